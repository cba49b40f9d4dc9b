/*
 * tad - evaluation of element-wise defined tensor expressions and of the
 * derivative expressions obtained by the element-wise derivation algorithm of
 * "Automatic Differentiation for Tensor Algebras" (Urban & van der Smagt, 2017).
 *
 * Model (Sec. 5.1 and Sec. 5.2 of the paper).  An output tensor f is defined
 * element by element,
 *
 *     f[alpha] = fbar( x^1[A^1 alpha_hat + o^1], ..., x^P[A^P alpha_hat + o^P] ),
 *
 * where alpha_hat = [alpha, k_1, ..., k_S] is the output multi-index extended by
 * the indices of the sums that occur inside the scalar function fbar, every A is
 * an integer matrix and every o an integer offset (the paper has o = 0; offsets
 * are an extension: beta is replaced by beta - o in every formula).  Given
 * df = dl/df the library evaluates, for every argument,
 *
 *     dx^p[beta] = delta(C (beta-o)) * sum_{z in Sigma(beta)} df[alpha] * d fbar / d x^p
 *                  at alpha_hat = I (beta-o) + K z                    (final equation of Sec. 5.1)
 *
 * with I, K, C from the Smith normal form of A (Sec. 4.1) and the summation
 * ranges Sigma from Fourier-Motzkin elimination (Sec. 4.2), as laid out in the
 * element-wise derivation algorithm of Sec. 5.3.
 *
 * Conventions
 *   - all tensors are float32, contiguous, row-major, zero-based (Sec. 6);
 *   - tad_compile / tad_plan_* are host-only and touch no GPU;
 *   - tad_forward / tad_backward take DEVICE pointers, enqueue work on the given
 *     CUDA stream (a cudaStream_t passed as void*, NULL = default stream), do not
 *     synchronise and allocate no device memory.  Passes of a call that are independent
 *     of each other (the zero fill of a gradient, a row or column sum beside a contraction)
 *     may run on a second stream that the plan owns (created by the first launch, released
 *     by tad_destroy); it is forked from and joined to the given stream with events, so
 *     the call is complete in the given stream's order and may be captured into a graph;
 *   - the caller owns every buffer; a plan's programs are immutable and the plan may be
 *     shared, but two host threads must not launch from the same plan at the same time
 *     (they would share that second stream's events);
 *   - every function returns a status; tad_last_error() gives a thread-local text.
 */
#ifndef TAD_INCLUDE_TAD_H
#define TAD_INCLUDE_TAD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tad_plan tad_plan;   /* opaque, owned by the library, freed by tad_destroy */

typedef enum {
    TAD_OK = 0,
    TAD_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, bad index */
    TAD_ERR_BAD_EXPR = 2,      /* malformed node list (order, operands, sum indices) */
    TAD_ERR_OUT_OF_RANGE = 3,  /* an index expression leaves its argument's shape */
    TAD_ERR_OVERFLOW = 4,      /* exact integer arithmetic left int64 / a tensor has >= 2^31 elements */
    TAD_ERR_UNSUPPORTED = 5,   /* valid but beyond the limits stated below */
    TAD_ERR_WORKSPACE = 6,     /* workspace too small or misaligned */
    TAD_ERR_CUDA = 7,          /* a CUDA runtime call failed; see tad_last_error() */
    TAD_ERR_NOMEM = 8
} tad_status;

/* Node operations of the scalar expression fbar: the elementary functions Sec. 2 builds its
 * computational graphs from (arithmetic, integer powers, exponential, logarithm, circular and
 * hyperbolic functions) and the sum over an index with a constant range of Sec. 5.2. */
typedef enum {
    TAD_OP_CONST = 0,   /* imm */
    TAD_OP_LOAD = 1,    /* element of an argument, through access[access] */
    TAD_OP_NEG = 2,
    TAD_OP_ADD = 3,
    TAD_OP_SUB = 4,
    TAD_OP_MUL = 5,
    TAD_OP_DIV = 6,
    TAD_OP_POWI = 7,    /* in0 ** ipow, literal integer exponent (the ** of Sec. 6) */
    TAD_OP_EXP = 8,
    TAD_OP_LOG = 9,
    TAD_OP_SIN = 10,
    TAD_OP_COS = 11,
    TAD_OP_TANH = 12,
    TAD_OP_SINH = 13,
    TAD_OP_COSH = 14,
    TAD_OP_SUM = 15     /* sum of in0 over alpha_hat[sum_idx] = sum_lo .. sum_hi (Sec. 5.2) */
} tad_op;

/* One index expression of one argument: x^arg[A alpha_hat + offset]  (Sec. 5.1). */
typedef struct {
    int32_t arg;             /* which tensor argument, 0 <= arg < n_args */
    const int64_t *A;        /* arg_rank[arg] x n_idx, row-major; n_idx = n_out_dims + n_sum_idx */
    const int64_t *offset;   /* arg_rank[arg] entries */
} tad_access;

typedef struct {
    int32_t op;              /* tad_op */
    int32_t in0, in1;        /* operand node ids (< own id), -1 if unused */
    int32_t access;          /* TAD_OP_LOAD: index into tad_expr.access */
    int32_t ipow;            /* TAD_OP_POWI */
    int32_t sum_idx;         /* TAD_OP_SUM: position of the sum's index in alpha_hat, >= n_out_dims */
    int64_t sum_lo, sum_hi;  /* TAD_OP_SUM: inclusive constant range (a convex integer set, Sec. 5.2) */
    double imm;              /* TAD_OP_CONST */
} tad_node;

typedef struct {
    int32_t n_out_dims;                 /* D_f */
    const int64_t *out_shape;           /* N^f */
    int32_t n_sum_idx;                  /* number of sum indices appended to alpha */
    int32_t n_args;                     /* P */
    const int32_t *arg_rank;            /* D_p */
    const int64_t *const *arg_shape;    /* N^p */
    int32_t n_access;
    const tad_access *access;
    int32_t n_nodes;
    const tad_node *nodes;              /* topological order, root last */
} tad_expr;

typedef struct {
    int32_t debug_bounds;   /* non-zero: kernels range-check every computed address, skip bad
                               accesses and record the first one (tad_debug_status) */
    int32_t saved_forward;  /* non-zero: the derivative kernels read the forward output f (as tad_forward wrote
                               it for the same arguments) wherever a derivative expression contains the value
                               of the whole expression, instead of evaluating it again.  Every backward entry
                               point then takes n_args + 1 pointers in `args`: the arguments, then f.  The
                               paper's algorithm keeps no values of the forward pass (Sec. 7); this option
                               is the usual trade of one |f|-sized read for the recomputation. */
    int32_t reserved[6];    /* must be zero */
} tad_options;

/* Limits: n_idx <= 8, argument rank <= 4, kernel dimension kappa <= 4, every tensor
 * < 2^31 elements, compiled program <= a few KB of bytecode (TAD_ERR_UNSUPPORTED beyond).
 * Every sum index belongs to exactly one sum node; a non-constant node must have one
 * set of enclosing sums on every path from the root. */
#define TAD_MAX_IDX 8
#define TAD_MAX_RANK 4
#define TAD_MAX_KAPPA 4
#define TAD_MAX_BOUND_ROWS 16

/*
 * tad_compile: the element-wise derivation algorithm of Sec. 5.3, once per expression.
 * For every index expression: Smith normal form of A restricted to the output indices and
 * the enclosing sum indices (Sec. 4.1; extended Euclid for the Bezout factors), cokernel /
 * pseudo-inverse / kernel, Fourier-Motzkin elimination of the box constraints written in
 * the kernel coordinates z (Sec. 4.2), scalar reverse-mode differentiation of fbar (Sec. 2)
 * and emission of bytecode for the forward and the derivative expressions.
 * opt may be NULL.  *out is written only on TAD_OK.  Host only.
 */
tad_status tad_compile(const tad_expr *expr, const tad_options *opt, tad_plan **out);

/* Frees a plan (NULL is allowed).  The caller makes sure no launch still uses it. */
void tad_destroy(tad_plan *plan);

/* Bytes of device workspace tad_forward and tad_backward need for this plan (may be 0).  The
 * workspace must be 256-byte aligned.  It holds the staged adjoints, the partial sums of
 * summations that are split over several thread blocks, the auxiliary tensors of the
 * expression optimisation (sums pushed inside the term: small pre-evaluated tensors and
 * contraction results, Sec. 6's clean-up step), and the debug word of a debug_bounds plan.
 * One workspace serves both calls; calls that share it must not overlap on the device. */
size_t tad_workspace_bytes(const tad_plan *plan);

/*
 * tad_forward: f[alpha] for every alpha of the output box (definition of an element-wise
 * specified function, Sec. 5.1; inner sums per Sec. 5.2).
 *   args       host array of n_args DEVICE pointers (read-only inputs), none NULL
 *   f          DEVICE pointer, prod(out_shape) floats, fully overwritten
 *   workspace  DEVICE pointer, tad_workspace_bytes() bytes, 256-byte aligned, caller-owned.  Only plans
 *              whose forward pass uses auxiliary tensors or a split summation read it; for every other
 *              plan NULL / 0 is accepted.  TAD_ERR_WORKSPACE when it is needed and missing or too small.
 */
tad_status tad_forward(const tad_plan *plan, const float *const *args, float *f,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * tad_backward: dx^p[beta] for every element of every requested argument, by the final
 * equation of Sec. 5.1 (gather form: one owner per output element, no atomics, fp32
 * accumulation); the results of several index expressions of one argument are added
 * (Sec. 5.3: dx <- 0, then accumulate over q).
 *   args   host array of n_args DEVICE pointers; for a plan compiled with saved_forward one more
 *          entry follows them: the forward output f of the same arguments (read-only), and the
 *          same holds for tad_backward_stage, tad_backward_arg and tad_backward_noalloc
 *   df     DEVICE pointer, prod(out_shape) floats
 *   dargs  host array of n_args DEVICE pointers; NULL entry = gradient not wanted;
 *          every requested tensor is fully overwritten (zeros where Gamma(beta) is empty)
 *   workspace  DEVICE pointer of at least tad_workspace_bytes() bytes (may be NULL if 0)
 */
tad_status tad_backward(const tad_plan *plan, const float *const *args, const float *df,
                        float *const *dargs, void *workspace, size_t workspace_bytes,
                        void *cuda_stream);

/*
 * The two halves of tad_backward, for callers that want gradients one at a time.
 * tad_backward_stage evaluates, once per output element, the adjoints of the top-level sums
 * that several gradients share (the factor df * d fbar / d s-bar of Sec. 5.2) into the
 * workspace; tad_backward_arg then evaluates the gradient of ONE argument and expects the
 * staged values of the same args / df to be in the workspace.  tad_backward is exactly
 * tad_backward_stage (when a requested gradient reads a staged value) followed by
 * tad_backward_arg for every requested argument.  The paper evaluates the derivative without
 * temporary memory (Sec. 7); staging trades |f| floats per staged sum for not repeating the
 * inner sum in every term.
 */
tad_status tad_backward_stage(const tad_plan *plan, const float *const *args, const float *df,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);
tad_status tad_backward_arg(const tad_plan *plan, const float *const *args, const float *df,
                            int32_t arg, float *darg, void *workspace, size_t workspace_bytes,
                            void *cuda_stream);

/*
 * tad_backward_noalloc: tad_backward for callers that cannot hand over a workspace because
 * they cannot allocate device memory themselves - for instance a plug-in called from inside
 * a host application's own memory pool, a callback that runs while allocation is forbidden,
 * or a process whose device-memory budget is fixed at start-up.  (The paper has no
 * counterpart: it evaluates derivatives without temporary memory, Sec. 7; this library
 * stages shared adjoints, keeps partial sums of split summations and the auxiliary tensors
 * of its expression optimisation in scratch.)
 *
 * The scratch is a fixed array of TAD_NOALLOC_SCRATCH_BYTES inside the library image; every
 * GPU that loads the library holds that much memory until the process exits.  A plan whose
 * tad_workspace_bytes() is larger is rejected with TAD_ERR_WORKSPACE and a message; nothing
 * is launched in that case.  The call allocates nothing (no cudaMalloc / cudaFree, no
 * allocating library routine); inputs and outputs are still the caller's buffers, with the
 * same meaning as in tad_backward.
 *
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.  All calls on one device share
 * the one array, which still holds whatever the previous call wrote: the entry point clears
 * the part that must start at zero (the debug word of debug_bounds plans) and overwrites the
 * rest before reading it, but two calls whose work overlaps on the GPU (different streams,
 * or different plans in flight at once) race on it and give wrong gradients.  Serialise them.
 */
#define TAD_NOALLOC_SCRATCH_BYTES (32u * 1024u * 1024u)
tad_status tad_backward_noalloc(const tad_plan *plan, const float *const *args, const float *df,
                                float *const *dargs, void *cuda_stream);

/*
 * tad_step_host: one forward and one backward pass with HOST buffers (same meaning as
 * tad_forward followed by tad_backward).  Inputs are copied to the device staging area,
 * results copied back.  The kernels run on the given stream, after whatever it already
 * holds; the copies run on two streams of the plan's own (created by the first call, released
 * by tad_destroy; calls on one plan must not run concurrently), ordered by events so
 * that df goes up during the forward pass and f and each gradient come down while the next
 * kernels run.  The call returns after all of it has drained.  Host buffers should be pinned for the copies to
 * be asynchronous.  staging is a DEVICE buffer of at least tad_staging_bytes() bytes,
 * 256-byte aligned, that the caller allocated; the library allocates nothing.  h_f and
 * entries of h_dargs may be NULL (not wanted).  (The paper has no counterpart; it is the
 * end-to-end entry point.)
 */
size_t tad_staging_bytes(const tad_plan *plan);
tad_status tad_step_host(const tad_plan *plan, const float *const *h_args, const float *h_df,
                         float *h_f, float *const *h_dargs,
                         void *staging, size_t staging_bytes, void *cuda_stream);

/* Text of the last non-OK status on the calling thread ("" if none). */
const char *tad_last_error(void);

/*
 * Measures the rate at which the current device retires FP32 multiply-adds from registers (a short kernel of
 * independent multiply-add chains, well under 100 ms, timed with events on the given stream; the call
 * synchronises).  The benchmark divides the algorithmic flops of ALU-bound kernels by this rate next to the
 * clock-derived peak.  No counterpart in the paper: a measurement aid.  Allocates four bytes for the duration
 * of the call.  *tflops is written only on TAD_OK.
 */
tad_status tad_measure_fp32_rate(void *cuda_stream, double *tflops);

/* debug_bounds plans: reads back (and clears) the debug word in `workspace` after
 * synchronising the stream.  TAD_ERR_OUT_OF_RANGE if a kernel skipped an out-of-range
 * access since the last query, TAD_OK otherwise.  workspace == NULL asks about the scratch
 * of tad_backward_noalloc on the current device (query it before the next call of that
 * entry point, which clears the word). */
tad_status tad_debug_status(const tad_plan *plan, void *workspace, void *cuda_stream);

/* ------------------------------------------------------------------------- */
/* Introspection (host only).  These are what the bit-exact plan tests use.   */
/* ------------------------------------------------------------------------- */

typedef struct {
    int32_t arg;                 /* argument this index expression reads */
    int32_t rank;                /* D_p: rows of A */
    int32_t n_idx;               /* columns of A-hat: output dims + enclosing sum indices */
    int32_t idx_pos[TAD_MAX_IDX];/* position in alpha_hat of each column */
    int32_t R;                   /* rank of A-hat (number of non-zero invariant factors) */
    int32_t kappa;               /* kernel dimension n_idx - R */
    int64_t A[TAD_MAX_RANK * TAD_MAX_IDX];      /* A-hat, rank x n_idx */
    int64_t offset[TAD_MAX_RANK];
    int64_t S[TAD_MAX_RANK];                    /* invariant factors alpha_1..alpha_R (Smith normal form) */
    int64_t U[TAD_MAX_RANK * TAD_MAX_RANK];     /* rank x rank, S = U A V; rows R.. are the cokernel C */
    int64_t V[TAD_MAX_IDX * TAD_MAX_IDX];       /* n_idx x n_idx; columns R.. are the kernel K in loop order */
    int64_t box_lo[TAD_MAX_IDX], box_hi[TAD_MAX_IDX];   /* inclusive range of every column's index */
    /* Bound rows of the kernel coordinates, loop 0 = outermost:
     *   ceil(max_r lower[r]) <= z_l <= floor(min_r upper[r]),
     *   row value = (c0 + sum_j cx[j]*x'_j + sum_{m<l} cz[m]*z_m) / den,  den > 0,
     * with x' = diag(1/alpha) U_R (beta - o). */
    int32_t n_lower[TAD_MAX_KAPPA], n_upper[TAD_MAX_KAPPA];
    int32_t masked;              /* 1 if a cokernel row or an invariant factor > 1 exists */
    int32_t lane_var;            /* which loop variable the kernel spreads over lanes */
} tad_access_info;

tad_status tad_plan_access_info(const tad_plan *plan, int32_t access, tad_access_info *out);

/* One bound row of loop `loop` (0 = outermost kernel coordinate) of an index expression.
 * upper = 0: lower-bound row, 1: upper-bound row.  coef_x has R entries, coef_z `loop` entries. */
tad_status tad_plan_bound_row(const tad_plan *plan, int32_t access, int32_t loop, int32_t upper,
                              int32_t row, int64_t *den, int64_t *c0, int64_t *coef_x, int64_t *coef_z);

/*
 * Enumerates Gamma-hat(beta) of one index expression on the host by walking the plan exactly
 * as the kernel does (mask, index transform, bound rows, nested ranges).  Writes up to `cap`
 * multi-indices alpha_hat (n_idx int64 each, in idx_pos order) and always the full count.
 */
tad_status tad_plan_enumerate(const tad_plan *plan, int32_t access, const int64_t *beta,
                              int64_t *alpha_hat_out, size_t cap, size_t *n_terms);

typedef struct {
    int64_t outputs;        /* elements written */
    int64_t terms;          /* sum over outputs of |Gamma-hat| (0 for the forward kernel) */
    double alg_bytes;       /* distinct elements read once + outputs written once, in bytes */
    double alg_flops;       /* each expression node once per distinct binding of the indices it depends on */
    double alg_transcendentals;
    int32_t bytecode_words; /* length of the program the interpreter runs */
    int32_t n_launches;     /* kernel launches this part issues */
} tad_kernel_stats;

/* Number of staged adjoints (|f| floats of workspace each). */
int32_t tad_plan_num_stages(const tad_plan *plan);

/* which = -1: forward kernel; which = q >= 0: backward kernel of index expression q;
 * which = -2 - s: staging kernel s. */
tad_status tad_plan_kernel_stats(const tad_plan *plan, int32_t which, tad_kernel_stats *out);

/* Human-readable listing of the compiled program (`which` as above); returns bytes needed. */
size_t tad_plan_disassemble(const tad_plan *plan, int32_t which, char *buf, size_t cap);

/*
 * The expression (which = -1) or the derived derivative through index expression `which` as text in the
 * notation of the listing in Sec. 6:
 *     f[i; j] = exp (-sum{k}_0^4 (...))
 *     dx[dx_0; dx_1] = if {conditions} then (sum{dx_z1}_lo^hi (sum{dx_z0}_lo^hi (term))) else (0)
 * Index positions of the term are written as their affine forms alpha = I beta + K z (Sec. 5.1); kernel
 * coordinates are named by kernel column (dx_z0, dx_z1, ...) and nested in the plan's loop order; ranges are the
 * bound rows of Sec. 4.2 (max [..] / min [..], with ceil / floor where a row does not divide); conditions are the
 * cokernel rows (= 0), divisibility by an invariant factor (mod n = 0, which the paper's listing never needs) and
 * guards (<= 0).  The kernel basis, and with it names and signs of the z, is the plan's: any unimodular
 * recombination describes the same set.  The text describes the derivative as derived, before the expression
 * clean-up that the kernels run.
 *   arg_names  n_args strings or NULL (x0, x1, ...);  idx_names  n_out_dims + n_sum_idx strings or NULL (i, j, k, ...)
 * Host only.  Returns the bytes needed including the terminator (0: no such expression); writes at most cap.
 */
size_t tad_plan_print(const tad_plan *plan, int32_t which, const char *const *arg_names, const char *const *idx_names,
                      char *buf, size_t cap);

/* Host-only pieces of Sec. 4, exported for tests.  Matrices are row-major int64. */
tad_status tad_extended_euclid(int64_t a, int64_t b, int64_t *gcd, int64_t *x, int64_t *y);
tad_status tad_smith_normal_form(const int64_t *A, int32_t n_rows, int32_t n_cols,
                                 int64_t *S, int64_t *U, int64_t *V, int32_t *rank);
/* Fourier-Motzkin elimination of  A z >= b  (b symbolic) in the order z_1 (eliminated first,
 * innermost loop) .. z_M (Algorithm of Sec. 4.2).  Per variable k the bounds are
 *   z_k >= (L b + L-hat z) / den   and   z_k <= (H b + H-hat z) / den
 * with integer rows and a positive denominator per row; F b <= 0 is the feasibility test.
 * Row r of variable k is stored at index k * cap_rows + r. */
tad_status tad_fourier_motzkin(const int64_t *A, int32_t n_rows, int32_t n_cols, int32_t cap_rows,
                               int32_t *n_lower, int32_t *n_upper,
                               int64_t *L_num, int64_t *Lhat_num, int64_t *L_den,
                               int64_t *H_num, int64_t *Hhat_num, int64_t *H_den,
                               int32_t *n_feas, int64_t *F_num);

#ifdef __cplusplus
}
#endif
#endif /* TAD_INCLUDE_TAD_H */

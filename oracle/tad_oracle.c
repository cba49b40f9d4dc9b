/*
 * CPU float64 oracle for element-wise defined tensor expressions and their
 * gradients.  TEST INFRASTRUCTURE ONLY: slow, plain and written to be checked
 * against the paper by eye.  It shares no code with the CUDA library and uses
 * none of the paper's symbolic derivation (no Smith normal form, no
 * Fourier-Motzkin elimination, no index inversion).
 *
 * What it computes:
 *   forward   f[alpha] = fbar(x^p[A alpha_hat + o], ...)            Sec. 5.1, Sec. 5.2
 *             a sum node loops its constant range and adds its body  (definition of s-bar, Sec. 5.2)
 *   backward  the "elementary approach" of Sec. 5.1 (the equation that sums
 *             over every alpha with a Kronecker delta on A alpha - beta),
 *             written in scatter form: for every alpha, walk the expression
 *             with the chain rule of Sec. 2 and add
 *                 df[alpha] * d fbar / d leaf
 *             into dx^p at the element that the leaf reads.
 *   counts    for one index expression: how many alpha_hat of the (sum-extended)
 *             box read each argument element, i.e. |Gamma-hat(beta)| of Sec. 5.2.
 *
 * Indices are zero-based (Sec. 6), tensors row-major and contiguous.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum {
    ON_CONST = 1, ON_LOAD, ON_NEG, ON_ADD, ON_SUB, ON_MUL, ON_DIV, ON_POWI,
    ON_EXP, ON_LOG, ON_SIN, ON_COS, ON_TANH, ON_SINH, ON_COSH, ON_SUM
};

enum { ORACLE_OK = 0, ORACLE_BAD_EXPR = 1, ORACLE_OUT_OF_RANGE = 2 };

#define ORACLE_MAX_IDX 16

typedef struct {
    int32_t op, in0, in1, access, ipow, sum_idx;
    int64_t sum_lo, sum_hi;
    double imm;
} oracle_node;

typedef struct {
    int32_t arg, rank;
    const int64_t *A;      /* rank x n_idx, row-major */
    const int64_t *off;    /* rank */
} oracle_access;

typedef struct {
    int32_t n_out_dims;
    const int64_t *out_shape;
    int32_t n_sum_idx;
    int32_t n_args;
    const int32_t *arg_rank;
    const int64_t *const *arg_shape;
    int32_t n_access;
    const oracle_access *access;
    int32_t n_nodes;
    const oracle_node *nodes;
} oracle_expr;

typedef struct {
    const oracle_expr *e;
    const double *const *args;
    int64_t ah[ORACLE_MAX_IDX];     /* current alpha_hat */
    int n_idx;
    int err;
    /* backward sinks */
    double *const *dx;
    double *const *tabs;
    int atomic;
} octx;

/* flat row-major position of the element that `access` reads at the current alpha_hat; -1 if outside */
static int64_t leaf_pos(octx *c, int q)
{
    const oracle_access *a = &c->e->access[q];
    const int64_t *shape = c->e->arg_shape[a->arg];
    int64_t flat = 0;
    for (int r = 0; r < a->rank; ++r) {
        int64_t b = a->off[r];
        for (int d = 0; d < c->n_idx; ++d) b += a->A[r * c->n_idx + d] * c->ah[d];
        if (b < 0 || b >= shape[r]) { c->err = ORACLE_OUT_OF_RANGE; return -1; }
        flat = flat * shape[r] + b;
    }
    return flat;
}

static double ipow_d(double x, int n)
{
    int m = n < 0 ? -n : n;
    double r = 1.0;
    for (int i = 0; i < m; ++i) r *= x;
    return n < 0 ? 1.0 / r : r;
}

/* value of node n at the current alpha_hat */
static double eval(octx *c, int n)
{
    const oracle_node *nd = &c->e->nodes[n];
    switch (nd->op) {
    case ON_CONST: return nd->imm;
    case ON_LOAD: {
        int64_t pos = leaf_pos(c, nd->access);
        return pos < 0 ? 0.0 : c->args[c->e->access[nd->access].arg][pos];
    }
    case ON_NEG:  return -eval(c, nd->in0);
    case ON_ADD:  return eval(c, nd->in0) + eval(c, nd->in1);
    case ON_SUB:  return eval(c, nd->in0) - eval(c, nd->in1);
    case ON_MUL:  return eval(c, nd->in0) * eval(c, nd->in1);
    case ON_DIV:  return eval(c, nd->in0) / eval(c, nd->in1);
    case ON_POWI: return ipow_d(eval(c, nd->in0), nd->ipow);
    case ON_EXP:  return exp(eval(c, nd->in0));
    case ON_LOG:  return log(eval(c, nd->in0));
    case ON_SIN:  return sin(eval(c, nd->in0));
    case ON_COS:  return cos(eval(c, nd->in0));
    case ON_TANH: return tanh(eval(c, nd->in0));
    case ON_SINH: return sinh(eval(c, nd->in0));
    case ON_COSH: return cosh(eval(c, nd->in0));
    case ON_SUM: {
        double acc = 0.0;
        for (int64_t k = nd->sum_lo; k <= nd->sum_hi; ++k) {
            c->ah[nd->sum_idx] = k;
            acc += eval(c, nd->in0);
        }
        return acc;
    }
    default: c->err = ORACLE_BAD_EXPR; return 0.0;
    }
}

/*
 * Chain rule (Sec. 2): `adj` is d f / d node along the path taken so far; a
 * node reached along several paths receives each path's contribution, which
 * adds up to the sum over consumers.  A sum node hands its adjoint unchanged
 * to its body at every k (d s-bar / d s = 1, Sec. 5.2).  At a leaf the term
 * df[alpha] * adj is scattered to the element the leaf reads.
 */
static void back(octx *c, int n, double adj, double df)
{
    const oracle_node *nd = &c->e->nodes[n];
    switch (nd->op) {
    case ON_CONST: return;
    case ON_LOAD: {
        int64_t pos = leaf_pos(c, nd->access);
        if (pos < 0) return;
        int p = c->e->access[nd->access].arg;
        double t = df * adj;
        if (c->dx[p]) {
            if (c->atomic) {
                #pragma omp atomic
                c->dx[p][pos] += t;
            } else c->dx[p][pos] += t;
        }
        if (c->tabs && c->tabs[p]) {
            double at = fabs(t);
            if (c->atomic) {
                #pragma omp atomic
                c->tabs[p][pos] += at;
            } else c->tabs[p][pos] += at;
        }
        return;
    }
    case ON_NEG: back(c, nd->in0, -adj, df); return;
    case ON_ADD: back(c, nd->in0, adj, df); back(c, nd->in1, adj, df); return;
    case ON_SUB: back(c, nd->in0, adj, df); back(c, nd->in1, -adj, df); return;
    case ON_MUL: {
        double u = eval(c, nd->in0), v = eval(c, nd->in1);
        back(c, nd->in0, adj * v, df);
        back(c, nd->in1, adj * u, df);
        return;
    }
    case ON_DIV: {
        double u = eval(c, nd->in0), v = eval(c, nd->in1);
        back(c, nd->in0, adj / v, df);
        back(c, nd->in1, -adj * u / (v * v), df);
        return;
    }
    case ON_POWI: {
        if (nd->ipow == 0) return;
        double u = eval(c, nd->in0);
        back(c, nd->in0, adj * (double)nd->ipow * ipow_d(u, nd->ipow - 1), df);
        return;
    }
    case ON_EXP:  back(c, nd->in0, adj * exp(eval(c, nd->in0)), df); return;
    case ON_LOG:  back(c, nd->in0, adj / eval(c, nd->in0), df); return;
    case ON_SIN:  back(c, nd->in0, adj * cos(eval(c, nd->in0)), df); return;
    case ON_COS:  back(c, nd->in0, -adj * sin(eval(c, nd->in0)), df); return;
    case ON_TANH: { double t = tanh(eval(c, nd->in0)); back(c, nd->in0, adj * (1.0 - t * t), df); return; }
    case ON_SINH: back(c, nd->in0, adj * cosh(eval(c, nd->in0)), df); return;
    case ON_COSH: back(c, nd->in0, adj * sinh(eval(c, nd->in0)), df); return;
    case ON_SUM:
        for (int64_t k = nd->sum_lo; k <= nd->sum_hi; ++k) {
            c->ah[nd->sum_idx] = k;
            back(c, nd->in0, adj, df);
        }
        return;
    default: c->err = ORACLE_BAD_EXPR; return;
    }
}

static int check_expr(const oracle_expr *e)
{
    if (!e || e->n_nodes <= 0 || e->n_out_dims < 0) return ORACLE_BAD_EXPR;
    if (e->n_out_dims + e->n_sum_idx > ORACLE_MAX_IDX) return ORACLE_BAD_EXPR;
    for (int n = 0; n < e->n_nodes; ++n) {
        const oracle_node *nd = &e->nodes[n];
        if (nd->op < ON_CONST || nd->op > ON_SUM) return ORACLE_BAD_EXPR;
        if (nd->in0 >= n || nd->in1 >= n) return ORACLE_BAD_EXPR;
        if (nd->op == ON_LOAD && (nd->access < 0 || nd->access >= e->n_access)) return ORACLE_BAD_EXPR;
        if (nd->op == ON_SUM && (nd->sum_idx < e->n_out_dims || nd->sum_idx >= e->n_out_dims + e->n_sum_idx))
            return ORACLE_BAD_EXPR;
    }
    return ORACLE_OK;
}

static int64_t box_count(const oracle_expr *e, const int64_t *lo, const int64_t *hi)
{
    int64_t n = 1;
    for (int d = 0; d < e->n_out_dims; ++d) n *= (hi[d] > lo[d] ? hi[d] - lo[d] : 0);
    return n;
}

/* decode the t-th multi-index of the sub-box [lo, hi) in row-major order; return flat position in f */
static int64_t decode(const oracle_expr *e, const int64_t *lo, const int64_t *hi, int64_t t, int64_t *alpha)
{
    for (int d = e->n_out_dims - 1; d >= 0; --d) {
        int64_t ext = hi[d] - lo[d];
        alpha[d] = lo[d] + t % ext;
        t /= ext;
    }
    int64_t flat = 0;
    for (int d = 0; d < e->n_out_dims; ++d) flat = flat * e->out_shape[d] + alpha[d];
    return flat;
}

/*
 * Forward pass over the sub-box lo <= alpha < hi of the output (the whole
 * output when lo = 0, hi = out_shape).  f and f_abs are full-size, only the
 * sub-box is written.  f_abs (may be NULL) receives the sum of |summands| when
 * the root is a sum node, |f| otherwise: the scale of the forward tolerance.
 */
int oracle_forward(const oracle_expr *e, const double *const *args,
                   const int64_t *lo, const int64_t *hi,
                   double *f, double *f_abs, int nthreads)
{
    int rc = check_expr(e);
    if (rc) return rc;
    const int root = e->n_nodes - 1;
    const int64_t total = box_count(e, lo, hi);
    int err = 0;
    if (nthreads < 1) nthreads = 1;
    #pragma omp parallel for schedule(static) num_threads(nthreads) reduction(|:err)
    for (int64_t t = 0; t < total; ++t) {
        octx c; memset(&c, 0, sizeof c);
        c.e = e; c.args = args; c.n_idx = e->n_out_dims + e->n_sum_idx;
        int64_t pos = decode(e, lo, hi, t, c.ah);
        f[pos] = eval(&c, root);
        if (f_abs) {
            const oracle_node *nd = &e->nodes[root];
            if (nd->op == ON_SUM) {
                double acc = 0.0;
                for (int64_t k = nd->sum_lo; k <= nd->sum_hi; ++k) {
                    c.ah[nd->sum_idx] = k;
                    acc += fabs(eval(&c, nd->in0));
                }
                f_abs[pos] = acc;
            } else f_abs[pos] = fabs(f[pos]);
        }
        err |= c.err;
    }
    return err;
}

/*
 * Backward pass in scatter form over the sub-box lo <= alpha < hi.  dx[p] and
 * t_abs[p] are full-size arrays that the CALLER has zeroed; a NULL entry skips
 * that argument.  t_abs[p] receives the sum of |terms| per element.  With
 * nthreads == 1 the order of additions is the row-major order of alpha and the
 * result is deterministic; with more threads additions are atomic and their
 * order is not fixed (float64, so the difference is far below any tolerance
 * used with fp32 data).
 */
int oracle_backward(const oracle_expr *e, const double *const *args, const double *df,
                    const int64_t *lo, const int64_t *hi,
                    double *const *dx, double *const *t_abs, int nthreads)
{
    int rc = check_expr(e);
    if (rc) return rc;
    const int root = e->n_nodes - 1;
    const int64_t total = box_count(e, lo, hi);
    int err = 0;
    if (nthreads < 1) nthreads = 1;
    #pragma omp parallel for schedule(static) num_threads(nthreads) reduction(|:err)
    for (int64_t t = 0; t < total; ++t) {
        octx c; memset(&c, 0, sizeof c);
        c.e = e; c.args = args; c.n_idx = e->n_out_dims + e->n_sum_idx;
        c.dx = dx; c.tabs = t_abs; c.atomic = nthreads > 1;
        int64_t pos = decode(e, lo, hi, t, c.ah);
        back(&c, root, 1.0, df[pos]);     /* d f / d f_1 = 1 (Sec. 2) */
        err |= c.err;
    }
    return err;
}

/* collect the sum nodes that enclose load nodes of `access` (same set required on every path) */
static int enclosing(const oracle_expr *e, int n, int access, int *stack, int depth,
                     int *found, int *set, int *nset)
{
    const oracle_node *nd = &e->nodes[n];
    if (nd->op == ON_LOAD) {
        if (nd->access != access) return ORACLE_OK;
        if (!*found) {
            *found = 1; *nset = depth;
            for (int i = 0; i < depth; ++i) set[i] = stack[i];
            return ORACLE_OK;
        }
        if (*nset != depth) return ORACLE_BAD_EXPR;
        for (int i = 0; i < depth; ++i) if (set[i] != stack[i]) return ORACLE_BAD_EXPR;
        return ORACLE_OK;
    }
    int rc = ORACLE_OK;
    if (nd->op == ON_SUM) {
        stack[depth] = n;
        return enclosing(e, nd->in0, access, stack, depth + 1, found, set, nset);
    }
    if (nd->in0 >= 0) rc |= enclosing(e, nd->in0, access, stack, depth, found, set, nset);
    if (nd->in1 >= 0) rc |= enclosing(e, nd->in1, access, stack, depth, found, set, nset);
    return rc;
}

/*
 * Term counts of one index expression: count[beta] = number of alpha_hat with
 * alpha in the sub-box, every enclosing sum index in its range, and
 * A alpha_hat + o = beta (the size of the sum-extended set of Sec. 5.2).
 * `count` is a full-size int64 array over the argument, zeroed by the caller.
 */
int oracle_counts(const oracle_expr *e, int access, const int64_t *lo, const int64_t *hi, int64_t *count)
{
    int rc = check_expr(e);
    if (rc) return rc;
    if (access < 0 || access >= e->n_access) return ORACLE_BAD_EXPR;
    int stack[ORACLE_MAX_IDX], set[ORACLE_MAX_IDX], nset = 0, found = 0;
    rc = enclosing(e, e->n_nodes - 1, access, stack, 0, &found, set, &nset);
    if (rc) return rc;
    if (!found) return ORACLE_OK;
    octx c; memset(&c, 0, sizeof c);
    c.e = e; c.n_idx = e->n_out_dims + e->n_sum_idx;
    const int64_t total = box_count(e, lo, hi);
    for (int64_t t = 0; t < total; ++t) {
        decode(e, lo, hi, t, c.ah);
        /* odometer over the enclosing sums */
        int64_t k[ORACLE_MAX_IDX];
        for (int s = 0; s < nset; ++s) k[s] = e->nodes[set[s]].sum_lo;
        int empty = 0;
        for (int s = 0; s < nset; ++s) if (e->nodes[set[s]].sum_hi < e->nodes[set[s]].sum_lo) empty = 1;
        while (!empty) {
            for (int s = 0; s < nset; ++s) c.ah[e->nodes[set[s]].sum_idx] = k[s];
            int64_t pos = leaf_pos(&c, access);
            if (pos >= 0) count[pos] += 1;
            int s = nset - 1;
            while (s >= 0) {
                if (++k[s] <= e->nodes[set[s]].sum_hi) break;
                k[s] = e->nodes[set[s]].sum_lo; --s;
            }
            if (s < 0) break;
        }
    }
    return c.err;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

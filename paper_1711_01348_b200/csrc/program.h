// Device program format: what the host compiler emits and the interpreter kernel runs.
// Plain structs, passed to the kernel BY VALUE (__grid_constant__), so the whole program
// sits in the constant bank and every fetch indexed by the (warp-uniform) program counter
// is a uniform constant load.
#pragma once
#include <stdint.h>

#define TADP_WARPS_PER_BLOCK 8
#define TADP_MAX_VARS 8       // loop variables of one kernel: outer + kernel coordinates + bound sums
#define TADP_MAX_CODE 320     // 8-byte instruction words
#define TADP_MAX_LOADS 20
#define TADP_MAX_LOOPS 8
#define TADP_MAX_ROWS 40      // bound rows + guard rows
#define TADP_MAX_PTRS 16      // arguments + df + staged adjoints + saved forward output
#define TADP_F_SLOT (TADP_MAX_PTRS - 1)   // pointer slot of the saved forward output (plans compiled with saved_forward)
#define TADP_MAX_DEPTH 8      // handlers are encoded for operand stack depths 0..7
#define TADP_NUM_TEMPS 8      // temporaries held in registers; further ones spill to local memory
#define TADP_MAX_SPILL 16
#define TADP_MAX_ZLOOPS 4     // kernel-coordinate loops per kernel
#define TADP_WIDE_DEPTH 4     // operand stack depth of the 16-element interpreter variant

// Interpreter operations.  The handler a word selects is op * 8 + k.  For operations on the
// operand stack k is the stack depth BEFORE the instruction, known to the host at emission
// time, so that every handler names its operand registers statically; for loop control k is
// the loop variable.
enum TadpOp : int {
    P_END = 0,
    // push one value (k = 0..6)
    P_CONST,      // imm (float bits)
    P_ZERO,       // 0 (accumulator of a value sum)
    P_LOAD,       // element-wise load through loads[a]
    P_LDT,        // temp[a]
    // replace the top (k = 1..7)
    P_NEG, P_SQR, P_CUBE,
    P_HSUM,       // top[t][u] <- sum over u' of top[t][u'] (closes a sum loop that runs over the element variable)
    P_MULC, P_ADDC,               // top <- top op imm(float)
    P_LDADD, P_LDMUL,             // top <- top op load(loads[a])
    P_LDADDSQ,                    // top <- (top + load(loads[a]))^2
    P_SCALE,      // acc <- acc * top ; pop (factors of the term that no loop variable touches, applied once)
    P_FN,         // top <- function b of top: TadpFn; F_POWI takes its exponent from imm; a != 0: the value is
                  // the same for every u, evaluate it once per lane-variable element
    P_STT,        // temp[a] <- top ; pop
    P_ACC,        // acc += active ? top : 0 ; pop
    // two operands (k = 2..7): second <- second op top ; pop
    P_ADD, P_SUB, P_MUL, P_DIV,
    P_SUMADD,     // second += top ; pop
    P_SUMEND,     // P_SUMADD followed by the P_SEND of loops[a] in one word
    P_FMAT,       // second <- second * temp[a] + top ; pop
    P_MACC,       // acc += active ? second * top : 0 ; pop 2
    // three operands (k = 3..7)
    P_FMA,        // third <- third * second + top ; pop 2
    // loop control (k = loop variable)
    P_SLOOP,      // bound sum loop begin: loops[a]; jumps to imm when the range is empty
    P_SEND,       // bound sum loop end: increments, jumps back to imm while in range
    P_USLOOP,     // the same for the sum whose index is the element variable: steps by UB, masks the tail
    P_USEND,
    P_ZLOOP,      // kernel-coordinate loop begin: loops[a]; computes the range from its bound rows
    P_ZEND,       // kernel-coordinate loop end
    P_XLOOP,      // every trip of an innermost loop in one word: runs bodies[imm] (a short accumulator program) and the
                  // loop end of loops[a]; follows the loop begin word; k = 1: the loop is a value sum whose accumulator
                  // is the bottom of the operand stack, k = 0: its terms go to the gradient accumulator.  In the
                  // 32-value shapes the body is a product of two loads (TadpBody::dot) and its steps are not read
    P_NUM_OPS
};

enum TadpFn : int { F_EXP = 0, F_LOG, F_SIN, F_COS, F_TANH, F_SINH, F_COSH, F_POWI };

struct alignas(8) TadpInsn {   // 8 bytes, fetched as one 64-bit constant load
    uint16_t handler;      // op * 8 + k
    uint8_t a, b;
    int32_t imm;
};

struct alignas(16) TadpLoad {         // 64 bytes, 16-byte aligned: 128-bit constant loads
    int32_t coef[TADP_MAX_VARS];       // element offset = base + sum_v coef[v] * var[v]  (mod 2^32)
    int32_t base;                      // constant element offset
    int32_t ptr;                       // which pointer slot (arguments first, then df, then staged adjoints)
    int32_t limit;                     // elements in the tensor (debug bounds)
    int32_t lane_step;                 // 32 * coef[lane variable]: offset step between vector elements
    int32_t rel_step;                  // coef[variable of the relative loop]
    int32_t unroll_step;               // coef[element variable]: offset step between elements u and u+1
    int32_t pad[2];
};

struct TadpRow {                       // value = (c0 + sum_v coef[v] * var[v]) / den, den > 0
    int32_t den;
    int32_t c0;
    int32_t coef[TADP_MAX_VARS];
};

struct TadpLoop {
    int32_t var;                       // loop variable it drives
    int32_t is_lane;                   // 1: spread over lanes and vector elements
    int32_t depends_on_lane;           // 1: some bound row reads the lane variable
    int32_t const_lo, const_hi;        // bound-sum loops: inclusive constant range
    int16_t lower0, n_lower;           // rows[lower0 .. lower0 + n_lower)
    int16_t upper0, n_upper;
    int32_t mask_level;                // position of its activity mask in the mask stack (1..)
    int32_t is_split;                  // 1: its range is divided into split_n contiguous shares; the warp with share
    int32_t split_n, split_div;        //    number s of an output takes share (s / split_div) % split_n
    int32_t is_relative;               // 1: every element walks its own short range, trip r visits lo_e + r
};

// Body of a fused innermost loop: an accumulator program over two value registers X and Y and up
// to two loop-invariant values I0, I1.  One byte per step, at most TADP_BODY_STEPS steps, 0 ends.
//   load step   1 kkk cc jj : v = load through slot jj fetched in manner kkk (TadpBodyFetch);
//                             cc = 0: X <- v, 1: X <- X + v, 2: X <- X * v, 3: X <- (X + v)^2
//   other steps 0 xxxxxxx   : TadpBodyStep
// After the steps the term goes to the sum:  TERM_X: S += X,  TERM_XY: S += Y * X.
#define TADP_BODY_STEPS 8
#define TADP_BODY_LOADS 4
#define TADP_MAX_BODIES 4
enum TadpBodyFetch : int { BF_EACH = 0, BF_ONE, BF_PER_T, BF_PER_U, BF_ROW };
enum TadpBodyStep : int {
    BS_END = 0, BS_PUSH,            // Y <- X
    BS_NEG, BS_SQR, BS_CUBE,        // X <- op X
    BS_ADDY, BS_SUBY, BS_MULY, BS_DIVY,   // X <- Y op X
    BS_LDI0, BS_LDI1,               // X <- I
    BS_MULI0, BS_MULI1, BS_ADDI0, BS_ADDI1,   // X <- X op I
    BS_FMAYI0, BS_FMAYI1            // X <- Y * I + X
};
enum TadpBodyLoopKind : int { BL_SUM = 0, BL_USUM, BL_Z, BL_Z_MASKED, BL_Z_LANE };
struct alignas(8) TadpBody {
    uint8_t steps[TADP_BODY_STEPS];
    uint8_t load[TADP_BODY_LOADS];     // load descriptor of every slot
    int32_t n_loads;
    int32_t loop_kind;                 // TadpBodyLoopKind
    int32_t term;                      // 0: S += X, 1: S += Y * X
    int32_t inv_kind[2];               // 0 unused, 1 constant (inv_value), 2 temporary (inv_value = its number)
    int32_t inv_value[2];
    // Product body: the term is the product of two loads and nothing else, S += P * Q with P = slot 0 and
    // Q = slot 1.  The 32-value shapes run only such bodies: P is fetched into a buffer of its shape
    // class (0: one value per u, 1: one per t), Q is multiplied in and accumulated as it arrives.
    int32_t dot;
    int32_t dot_pclass;
    int32_t dot_fk[2];                 // TadpBodyFetch of P and Q
};

struct alignas(16) TadpProgram {
    int32_t n_code, n_loads, n_loops, n_rows;
    int32_t n_outer;                   // outer variables 0 .. n_outer-1 (decoded from the work item)
    int32_t lane_var;                  // variable A spread over lanes (and elements t); < n_outer: distinct outputs per lane
    int32_t unroll_var;                // variable B spread over the elements u of each thread, or -1
    int32_t unroll_kind;               // 0 none, 1 outer variable (distinct outputs per u), 3 bound sum
    int32_t outer_lo[TADP_MAX_VARS];   // inclusive box of the outer variables
    int32_t outer_ext[TADP_MAX_VARS];  // extents (>= 1)
    int32_t n_guards, guard0;          // rows[guard0 ..): element is live iff every row value <= 0 (den = 1)
    int32_t out_base;                  // output element offset = out_base + sum_v out_coef[v] * var[v]
    int32_t out_coef[TADP_MAX_VARS];
    int32_t out_limit;
    int32_t accumulate;                // 0: out = acc ; 1: out += acc
    int32_t write_only_live;           // 1: skip elements whose Gamma is empty (output pre-zeroed)
    int32_t zsplit;                    // > 1: that many warps share every output; each writes a partial sum
    int32_t rel_var;                   // variable of the relative loop, or -1
    int32_t part_coef[TADP_MAX_VARS];  // zsplit > 1: compact index of an output in its plane of partial sums,
    int32_t part_limit;                //   sum_v part_coef[v] * (var[v] - outer_lo[v]); part_limit entries per plane
    TadpInsn code[TADP_MAX_CODE];
    TadpLoad loads[TADP_MAX_LOADS];
    TadpLoop loops[TADP_MAX_LOOPS];
    TadpRow rows[TADP_MAX_ROWS];
    int32_t n_bodies;
    TadpBody bodies[TADP_MAX_BODIES];
};

struct TadpPointers {
    const float *in[TADP_MAX_PTRS];
    float *out;
    float *part;                       // zsplit > 1: zsplit planes of part_limit partial sums, then one plane of
                                       // flags (non-zero: some share of that output accumulated a term)
    int32_t *debug;                    // NULL unless the plan was compiled with debug_bounds
};

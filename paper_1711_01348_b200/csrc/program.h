// Device program format: what the host compiler emits and the interpreter kernel runs.
// Plain structs, passed to the kernel BY VALUE (__grid_constant__), so the whole program
// sits in the constant bank and every fetch indexed by the (warp-uniform) program counter
// is a uniform constant load.
#pragma once
#include <stdint.h>

#define TADP_MAX_VARS 8       // loop variables of one kernel: outer + kernel coordinates + bound sums
#define TADP_MAX_CODE 320     // 8-byte instruction words
#define TADP_MAX_LOADS 20
#define TADP_MAX_LOOPS 8
#define TADP_MAX_ROWS 40      // bound rows + guard rows
#define TADP_MAX_PTRS 8       // arguments + df
#define TADP_MAX_DEPTH 8      // handlers are encoded for operand stack depths 0..7
#define TADP_NUM_TEMPS 8      // temporaries held in registers; further ones spill to local memory
#define TADP_MAX_SPILL 16
#define TADP_MAX_ZLOOPS 4     // kernel-coordinate loops per kernel

// Interpreter operations.  The handler a word selects is op * TADP_MAX_DEPTH + d where d is
// the operand stack depth BEFORE the instruction, known to the host at emission time; this
// lets every handler name its operand registers statically.
enum TadpOp : int {
    P_END = 0,
    P_CONST,      // push imm (float bits)
    P_LOAD,       // push element-wise load through loads[a]
    P_NEG, P_EXP, P_LOG, P_SIN, P_COS, P_TANH, P_SINH, P_COSH,
    P_SQR,        // top <- top^2
    P_POWI,       // top <- top ** imm (signed integer)
    P_ADD, P_SUB, P_MUL, P_DIV,   // second <- second op top ; pop
    P_MULC, P_ADDC,               // top <- top op imm(float)
    P_FMA,        // third <- third * second + top ; pop 2
    P_LDT,        // push temp[a]
    P_STT,        // temp[a] <- top ; pop
    P_ZERO,       // push 0 (accumulator of a value sum)
    P_SUMADD,     // second += top ; pop
    P_SLOOP,      // bound sum loop begin: loops[a]; jumps to imm when the range is empty
    P_SEND,       // bound sum loop end: increments, jumps back to imm while in range
    P_ZLOOP,      // kernel-coordinate loop begin: loops[a]; computes the range from its bound rows
    P_ZEND,       // kernel-coordinate loop end
    P_ACC,        // acc += active ? top : 0 ; pop
    P_NUM_OPS
};

struct TadpInsn {          // 8 bytes
    uint16_t handler;      // op * TADP_MAX_DEPTH + depth
    uint8_t a, b;
    int32_t imm;
};

struct TadpLoad {
    int32_t ptr;                       // which pointer slot (arguments first, then df)
    int32_t base;                      // constant element offset
    int32_t coef[TADP_MAX_VARS];       // element offset = base + sum_v coef[v] * var[v]  (mod 2^32)
    int32_t limit;                     // elements in the tensor (debug bounds)
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
    int32_t mask_level;                // position of its activity mask in the mask word (1..)
};

struct TadpProgram {
    int32_t n_code, n_loads, n_loops, n_rows;
    int32_t n_outer;                   // outer variables 0 .. n_outer-1 (decoded from the work item)
    int32_t lane_var;                  // variable spread over lanes; < n_outer: distinct outputs per lane
    int32_t outer_lo[TADP_MAX_VARS];   // inclusive box of the outer variables
    int32_t outer_ext[TADP_MAX_VARS];  // extents (>= 1)
    int32_t n_guards, guard0;          // rows[guard0 ..): element is live iff every row value <= 0 (den = 1)
    int32_t out_base;                  // output element offset = out_base + sum_v out_coef[v] * var[v]
    int32_t out_coef[TADP_MAX_VARS];
    int32_t out_limit;
    int32_t accumulate;                // 0: out = acc ; 1: out += acc
    int32_t write_only_live;           // 1: skip elements whose Gamma is empty (output pre-zeroed)
    TadpInsn code[TADP_MAX_CODE];
    TadpLoad loads[TADP_MAX_LOADS];
    TadpLoop loops[TADP_MAX_LOOPS];
    TadpRow rows[TADP_MAX_ROWS];
};

struct TadpPointers {
    const float *in[TADP_MAX_PTRS];
    float *out;
    int32_t *debug;                    // NULL unless the plan was compiled with debug_bounds
};

// Element-wise programs: kernels without loops, run by tad_ew_kernel (ew.cu).
// An accumulator program over two value registers X and Y; every step acts on the four consecutive
// outputs of a thread.  After the last step X is stored.
#pragma once
#include <stdint.h>

#include "program.h"

enum TadeOp : int {
    E_END = 0,
    E_LD,        // v = load through loads[a];  b = 0: X <- v, 1: X <- X + v, 2: X <- X * v, 3: X <- (X + v)^2
    E_PUSH,      // Y <- X
    E_CONST,     // X <- imm
    E_NEG, E_SQR, E_CUBE,
    E_MULC, E_ADDC,              // X <- X op imm
    E_ADDY, E_SUBY, E_MULY, E_DIVY,   // X <- Y op X
    E_FN         // X <- function b (TadpFn) of X; a = exponent of F_POWI
};

struct TadeStep { uint8_t op, b; int16_t a; float imm; };

#define TADE_MAX_STEPS 24
#define TADE_MAX_LOADS 8

struct alignas(16) TadeProgram {
    int32_t n_outer, lane_var;                 // the lane variable is the one along which the output is contiguous
    int32_t outer_lo[TADP_MAX_VARS], outer_ext[TADP_MAX_VARS];
    uint32_t div_mul[TADP_MAX_VARS];           // n / outer_ext[v] = (n * div_mul[v]) >> div_shift[v] for n < 2^31
    int32_t div_shift[TADP_MAX_VARS];
    int32_t out_base, out_coef[TADP_MAX_VARS], out_limit, accumulate;
    int32_t n_loads, n_steps;
    TadpLoad loads[TADE_MAX_LOADS];
    TadeStep steps[TADE_MAX_STEPS];
};

// Line-sum programs: the final sum of Sec. 5.1 for a term that is a product of index expressions,
//     out[beta] = scale(beta) * sum over z of  c * L_1[..] * L_2[..] * ...,
// with one or two summation loops whose bounds are the integer rows of Sec. 4.2 (true floor / ceiling,
// evaluated once per loop run).  Run by tad_line_kernel (line.cu) without interpretation: a thread (or a
// warp) owns an output, walks its ranges and multiplies the loads of every term.
#pragma once
#include <stdint.h>

#include "program.h"

#define TADL_MAX_LOADS 4
#define TADL_MAX_ROWS 6

struct TadlLoad { int32_t ptr, base; int32_t coef[TADP_MAX_VARS]; int32_t cz[2]; int32_t sq; };     // offset = base + coef . outer + cz . z; sq: the value enters squared
struct TadlRow { int32_t den, c0; int32_t coef[TADP_MAX_VARS]; int32_t cz; };           // (c0 + coef . outer + cz * z0) / den

struct alignas(16) TadlProgram {
    int32_t n_outer, lane_var;
    int32_t mode;                          // 0: a thread per output, lanes along lane_var; 1: a warp per output, lanes along the inner loop
    int32_t outer_lo[TADP_MAX_VARS], outer_ext[TADP_MAX_VARS];
    uint32_t div_mul[TADP_MAX_VARS]; int32_t div_shift[TADP_MAX_VARS];     // multiply-shift division by outer_ext
    int32_t n_loops;                       // 1 or 2 (loop 0 outermost; the rows of loop 1 may read z0)
    int32_t n_lower[2], n_upper[2];
    TadlRow lower[2][TADL_MAX_ROWS], upper[2][TADL_MAX_ROWS];
    int32_t n_guards; TadlRow guards[TADL_MAX_ROWS];                       // live iff every value <= 0 (den = 1)
    int32_t n_loads; TadlLoad loads[TADL_MAX_LOADS];
    float cterm;
    int32_t n_scale; TadlLoad scale[2]; float cscale;                      // factor outside the sums: cscale * product
    int32_t out_base, out_coef[TADP_MAX_VARS], out_limit, accumulate;
    int32_t zsplit;                        // > 1: grid.y shares, each writing a plane of partial sums; share = s0 * n_share[1] + s1
    int32_t n_share[2], chunk_shift[2], zbox_lo[2];
    // the box of loop l is cut into pieces of 2^chunk_shift values counted from zbox_lo; share s_l of an output walks the
    // s_l-th piece counted from the one its range starts in (cut to the range), so that neighbouring outputs stay in step
    int32_t part_limit, part_coef[TADP_MAX_VARS];
    int32_t stream;                        // load 0 is consecutive along the lanes: read with evict-first loads
    int32_t unroll;                        // terms a thread keeps in flight: 2, 4 or 8
    int32_t live_plane;                    // share 0 also writes plane zsplit: 1 where the guards hold (outputs of masked gradients that exist)
};

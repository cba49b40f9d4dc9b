// Contraction programs: what the host emits for a kernel whose term is a product of two index
// expressions summed over loop variables that both of them (or one of them) read,
//
//     out[m, n] (+)= scale * sum_k  A[m, k] * B[n, k]
//
// which is the final sum of Sec. 5.1 (and the sum of Sec. 5.2 in the forward direction) for a
// product body; the matrix product f^4 of Sec. 5 is the smallest instance.  m, n, k (and a batch
// index z) are flattened groups of loop variables in mixed radix; because every index expression is
// affine, the element offset of an operand splits into a part per group, which is what the tile
// kernel exploits: it gathers a tile of each operand into shared memory with offsets
// row_part(m) + k_part(k) and runs a register-tiled multiply-add loop over it.
#pragma once
#include <stdint.h>

#define TADC_MAX_DIGITS 4
#define TADC_BK 32            // summation indices per shared-memory stage

struct TadcGroup {             // flattened index group, last digit fastest
    int32_t n_digits;
    int32_t extent;            // product of ext[]
    int32_t ext[TADC_MAX_DIGITS];
    int32_t sA[TADC_MAX_DIGITS];   // element stride of every digit in operand A, operand B, the output
    int32_t sB[TADC_MAX_DIGITS];
    int32_t sO[TADC_MAX_DIGITS];
    int32_t gA[TADC_MAX_DIGITS];   // coefficient of every digit in the guard expression of A and of B
    int32_t gB[TADC_MAX_DIGITS];
};

// how a tile of an operand is gathered
enum TadcGather : int {
    TG_ROW = 0,    // lanes along the row index (m or n), 4 bytes per copy
    TG_K,          // lanes along the summation index, 4 bytes per copy
    TG_ROW16       // rows contiguous and 16-byte aligned: 16 bytes per copy along the row index
};

// steps applied to every finished sum before it is stored (in this order)
enum TadcEpilogueOp : int { TE_END = 0, TE_NEG, TE_EXP, TE_MULC, TE_ADDC, TE_MUL_LOAD, TE_ADD_LOAD, TE_SQR, TE_TANH, TE_SIN, TE_COS };
#define TADC_MAX_EPI 6

struct alignas(16) TadcProgram {
    TadcGroup M, N, K, Z;
    int32_t ptrA, ptrB;            // pointer slots of the operands; ptrB < 0: B is all ones (a plain summation of A)
    int32_t baseA, baseB, baseO;   // constant element offsets
    // an operand element is read as zero unless 0 <= c0 + sum(g * digit) < ext (guard = 1), always read when guard = 0
    int32_t guardA, guardA_c0, guardA_ext;
    int32_t guardB, guardB_c0, guardB_ext;
    int32_t modeA, modeB;          // TadcGather
    int32_t ksplit;                // > 1: the summation range is divided into that many chunks, one plane of partial sums each
    int32_t kchunk;                // summation indices per chunk (a multiple of TADC_BK)
    int32_t accumulate;            // 1: out += result
    int32_t out_vec4;              // 1: four consecutive n are four consecutive, 16-byte aligned output elements
    int32_t shape;                 // tiles: 0 = 128 x 128 (8 x 8 per thread), 1 = 128 x 32, 2 = 128 x 64, 3 = 128 x 36 (8 x 4 per thread);
                                   // 4 = sums of rows (a warp per output), 5 = streamed narrow contraction, 6 = sums of columns (a thread per output)
    float scale;
    int32_t n_epi;
    int32_t epi_op[TADC_MAX_EPI];
    float epi_imm[TADC_MAX_EPI];
    int32_t epi_ptr[TADC_MAX_EPI]; // TE_*_LOAD: pointer slot; the element is read at epi_base + the offset of the output element
    int32_t epi_base[TADC_MAX_EPI];
};

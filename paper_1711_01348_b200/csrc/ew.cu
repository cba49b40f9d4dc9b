// Element-wise kernel: programs without loops (forward passes of expressions without sums, function
// tables, operand matrices of contractions, the element-wise remainder of a factored kernel).
//
// The program is a short accumulator program over two value registers X and Y (ew.h), every step
// dispatched once for the four consecutive outputs a thread owns along the output's contiguous
// variable; a thread block covers a tile of rows x 4-element columns chosen so that short rows still
// fill the block.  Index arithmetic: the row number is split into the outer variables with
// multiply-shift divisions prepared by the host, every load's offset is its affine form in those
// variables.  Loads whose offset steps by +1 along the row and are 16-byte aligned are 128-bit loads,
// loads that do not move along the row are read once; the store is one 128-bit store.
#include <cuda_runtime.h>

#include <algorithm>

#include "ew.h"
#include "vm.cuh"

namespace {

using tadvm::apply_fn;
using tadvm::fast_sincos;
using tadvm::fast_tanh;

constexpr int EG = 4;          // groups of four consecutive outputs per thread, one block-wide row segment apart

__global__ void __launch_bounds__(256)
tad_ew_kernel(const __grid_constant__ TadeProgram P, const __grid_constant__ TadpPointers ptrs, const unsigned n_items,
              const unsigned cols, const unsigned lane_blocks, const unsigned n_rows)
{
    const unsigned tid = threadIdx.x;
    const unsigned rows_per_block = 256u / cols;
    const unsigned tc = tid % cols, tr = tid / cols;
    const int lane_var = P.lane_var;
    const unsigned lane_ext = (unsigned)P.outer_ext[lane_var];
    const unsigned gstride = cols * 4u;                       // elements between two groups of a thread
    const bool few_vars = P.n_outer <= 4;
    for (unsigned item = blockIdx.x; item < n_items; item += gridDim.x) {
        const unsigned lb = item % lane_blocks, rb = item / lane_blocks;
        const unsigned row = rb * rows_per_block + tr, lane0 = lb * gstride * EG + tc * 4u;
        if (row >= n_rows || lane0 >= lane_ext) continue;
        int live[EG];
#pragma unroll
        for (int g = 0; g < EG; ++g) { const unsigned l = lane0 + g * gstride; live[g] = l >= lane_ext ? 0 : (int)min(4u, lane_ext - l); }
        // outer variables of this row (the lane variable holds the first of the thread's elements)
        int var[TADP_MAX_VARS];
        unsigned rem = row;
#pragma unroll
        for (int v = TADP_MAX_VARS - 1; v >= 0; --v) {
            var[v] = 0;
            if (v < P.n_outer) {
                if (v == lane_var) var[v] = P.outer_lo[v] + (int)lane0;
                else {
                    const unsigned q = (unsigned)(((unsigned long long)rem * (unsigned)P.div_mul[v]) >> P.div_shift[v]);
                    var[v] = P.outer_lo[v] + (int)(rem - q * (unsigned)P.outer_ext[v]);
                    rem = q;
                }
            }
        }
        // offset = base + coef . var (the variables stay in registers: every index below is a compile-time constant)
#define TAD_EW_AFFINE(off, coef, base)                                                                   \
    unsigned off = (unsigned)(base);                                                                       \
    if (few_vars) { _Pragma("unroll") for (int v = 0; v < 4; ++v) off += (unsigned)(coef)[v] * (unsigned)var[v]; } \
    else { _Pragma("unroll") for (int v = 0; v < TADP_MAX_VARS; ++v) off += (unsigned)(coef)[v] * (unsigned)var[v]; }
        float X[EG][4], Y[EG][4];
#pragma unroll
        for (int g = 0; g < EG; ++g)
#pragma unroll
            for (int j = 0; j < 4; ++j) { X[g][j] = 0.f; Y[g][j] = 0.f; }
#define TAD_EW_ALL(expr)                                                \
    _Pragma("unroll") for (int g = 0; g < EG; ++g)                       \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) { expr; }
        for (int s = 0; s < P.n_steps; ++s) {
            const TadeStep st = P.steps[s];
            switch (st.op) {
            case E_LD: {
                const TadpLoad &L = P.loads[st.a];
                TAD_EW_AFFINE(off0, L.coef, L.base)
                const int step = L.coef[lane_var];
                const float *__restrict__ src = ptrs.in[L.ptr];
                const bool wide = step == 1 && ((off0 & 3u) == 0) && ((reinterpret_cast<uintptr_t>(src) & 15u) == 0);
                const float first = step == 0 ? __ldg(src + off0) : 0.f;
#pragma unroll
                for (int g = 0; g < EG; ++g) {
                    float v4[4];
                    const unsigned off = (unsigned)((int)off0 + g * (int)gstride * step);
                    if (step == 0) { v4[0] = v4[1] = v4[2] = v4[3] = first; }
                    else if (wide && live[g] == 4) {
                        const float4 q = __ldg(reinterpret_cast<const float4 *>(src + off));
                        v4[0] = q.x; v4[1] = q.y; v4[2] = q.z; v4[3] = q.w;
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) v4[j] = j < live[g] ? __ldg(src + (unsigned)((int)off + j * step)) : 0.f;
                    }
                    if (st.b == 0) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) X[g][j] = v4[j];
                    } else if (st.b == 1) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) X[g][j] += v4[j];
                    } else if (st.b == 2) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) X[g][j] *= v4[j];
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) { const float t = X[g][j] + v4[j]; X[g][j] = t * t; }
                    }
                }
                break;
            }
            case E_PUSH: TAD_EW_ALL(Y[g][j] = X[g][j]) break;
            case E_CONST: TAD_EW_ALL(X[g][j] = st.imm) break;
            case E_NEG: TAD_EW_ALL(X[g][j] = -X[g][j]) break;
            case E_SQR: TAD_EW_ALL(X[g][j] *= X[g][j]) break;
            case E_CUBE: TAD_EW_ALL(X[g][j] = X[g][j] * X[g][j] * X[g][j]) break;
            case E_MULC: TAD_EW_ALL(X[g][j] *= st.imm) break;
            case E_ADDC: TAD_EW_ALL(X[g][j] += st.imm) break;
            case E_ADDY: TAD_EW_ALL(X[g][j] = Y[g][j] + X[g][j]) break;
            case E_SUBY: TAD_EW_ALL(X[g][j] = Y[g][j] - X[g][j]) break;
            case E_MULY: TAD_EW_ALL(X[g][j] = Y[g][j] * X[g][j]) break;
            case E_DIVY: TAD_EW_ALL(X[g][j] = Y[g][j] / X[g][j]) break;
            case E_FN:
                // (every loop over the values is fully unrolled: X and Y must stay in registers)
                switch (st.b) {
                case F_EXP: TAD_EW_ALL(X[g][j] = __expf(X[g][j])) break;
                case F_TANH: TAD_EW_ALL(X[g][j] = fast_tanh(X[g][j])) break;
                case F_SIN: TAD_EW_ALL(X[g][j] = fabsf(X[g][j]) < 8192.f ? fast_sincos(X[g][j], 0) : apply_fn(F_SIN, X[g][j], 0)) break;
                case F_COS: TAD_EW_ALL(X[g][j] = fabsf(X[g][j]) < 8192.f ? fast_sincos(X[g][j], 1) : apply_fn(F_COS, X[g][j], 0)) break;
                default: TAD_EW_ALL(X[g][j] = apply_fn(st.b, X[g][j], st.a)) break;
                }
                break;
            default: break;
            }
        }
#undef TAD_EW_ALL
        float *__restrict__ out = ptrs.out;
        const int ostep = P.out_coef[lane_var];
        TAD_EW_AFFINE(out0, P.out_coef, P.out_base)
        const bool wide_out = ostep == 1 && ((out0 & 3u) == 0) && ((reinterpret_cast<uintptr_t>(out) & 15u) == 0);
#pragma unroll
        for (int g = 0; g < EG; ++g) {
            const unsigned out_off = (unsigned)((int)out0 + g * (int)gstride * ostep);
            if (wide_out && live[g] == 4) {
                float4 *dst = reinterpret_cast<float4 *>(out + out_off);
                float4 r = make_float4(X[g][0], X[g][1], X[g][2], X[g][3]);
                if (P.accumulate) { const float4 o = *dst; r.x += o.x; r.y += o.y; r.z += o.z; r.w += o.w; }
                *dst = r;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < live[g]) { const unsigned o = (unsigned)((int)out_off + j * ostep); out[o] = P.accumulate ? out[o] + X[g][j] : X[g][j]; }
            }
        }
#undef TAD_EW_AFFINE
    }
}

}  // namespace

cudaError_t tad_launch_ew(const TadeProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream)
{
    const unsigned lane_ext = (unsigned)P.outer_ext[P.lane_var];
    unsigned long long rows = 1;
    for (int v = 0; v < P.n_outer; ++v) if (v != P.lane_var) rows *= (unsigned long long)P.outer_ext[v];
    if (lane_ext == 0 || rows == 0) return cudaSuccess;
    unsigned cols = 1;
    while (cols < 256u && cols * 4u * EG < lane_ext) cols *= 2u;
    const unsigned rows_per_block = 256u / cols;
    const unsigned lane_blocks = (lane_ext + cols * 4u * EG - 1u) / (cols * 4u * EG);
    const unsigned long long row_blocks = (rows + rows_per_block - 1) / rows_per_block;
    const unsigned long long items = row_blocks * lane_blocks;
    if (items >= (1ull << 32) || rows >= (1ull << 31)) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)std::min<unsigned long long>(items, (unsigned long long)sms * 16ull);
    tad_ew_kernel<<<grid, 256, 0, stream>>>(P, ptrs, (unsigned)items, cols, lane_blocks, (unsigned)rows);
    return cudaGetLastError();
}

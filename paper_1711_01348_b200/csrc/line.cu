// Kernel for line-sum programs (line.h).  No atomics: a split range writes planes of partial sums that the
// fixed-order reduction of the interpreter adds.
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>

#include "line.h"

namespace {

__device__ __forceinline__ int fdiv(int a, int b) { int q = a / b; return (a % b != 0 && a < 0) ? q - 1 : q; }
__device__ __forceinline__ int cdiv(int a, int b) { int q = a / b; return (a % b != 0 && a > 0) ? q + 1 : q; }

template <int V>
__device__ __forceinline__ int row_num(const TadlRow &r, const int (&var)[V], int z0)
{
    int n = r.c0 + r.cz * z0;
#pragma unroll
    for (int v = 0; v < V; ++v) n += r.coef[v] * var[v];
    return n;
}

// [lo, hi] of loop l for this output (and this z0)
template <int V>
__device__ __forceinline__ void range(const TadlProgram &P, int l, const int (&var)[V], int z0, int &lo, int &hi)
{
    lo = INT_MIN; hi = INT_MAX;
    for (int r = 0; r < P.n_lower[l]; ++r) { const TadlRow &R = P.lower[l][r]; const int n = row_num(R, var, z0); lo = max(lo, R.den == 1 ? n : cdiv(n, R.den)); }
    for (int r = 0; r < P.n_upper[l]; ++r) { const TadlRow &R = P.upper[l][r]; const int n = row_num(R, var, z0); hi = min(hi, R.den == 1 ? n : fdiv(n, R.den)); }
}

constexpr int V = 4;     // outer variables a line-sum program may have

// One run of the innermost loop: sum over z = z0, z0 + step, ... <= hi of the product of NL loads, every offset advancing
// by its own constant.  U terms are in flight at once (their loads are issued before the first multiplication), each
// with its own accumulator; the accumulators are added in a fixed order at the end.  Where load 0 (the largest
// operand) is consecutive along the lanes every line of it is used once: it then streams through the cache (evict-first)
// and leaves the lines of the smaller operands alone.
template <int NL, int U, bool STREAM>
__device__ __forceinline__ float walk(const float *const (&src)[4], const int (&sq)[4], int (&o)[4], const int (&d)[4], int z, const int hi, const int step)
{
    float s[U];
#pragma unroll
    for (int u = 0; u < U; ++u) s[u] = 0.f;
    for (; z + (U - 1) * step <= hi; z += U * step) {
        float v[U][NL];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int l = 0; l < NL; ++l) v[u][l] = (l == 0 && STREAM) ? __ldcs(src[l] + (unsigned)(o[l] + u * d[l])) : __ldg(src[l] + (unsigned)(o[l] + u * d[l]));
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float p = sq[0] ? v[u][0] * v[u][0] : v[u][0];
#pragma unroll
            for (int l = 1; l < NL; ++l) p *= sq[l] ? v[u][l] * v[u][l] : v[u][l];
            s[u] += p;
        }
#pragma unroll
        for (int l = 0; l < NL; ++l) o[l] += U * d[l];
    }
    for (; z <= hi; z += step) {
        float p = STREAM ? __ldcs(src[0] + (unsigned)o[0]) : __ldg(src[0] + (unsigned)o[0]);
        if (sq[0]) p *= p;
#pragma unroll
        for (int l = 1; l < NL; ++l) { const float x = __ldg(src[l] + (unsigned)o[l]); p *= sq[l] ? x * x : x; }
        s[0] += p;
#pragma unroll
        for (int l = 0; l < NL; ++l) o[l] += d[l];
    }
    float total = 0.f;
#pragma unroll
    for (int u = 0; u < U; ++u) total += s[u];
    return total;
}

template <bool STREAM>
__global__ void __launch_bounds__(256)
tad_line_kernel(const __grid_constant__ TadlProgram P, const __grid_constant__ TadpPointers ptrs, const unsigned n_items,
                const unsigned cols, const unsigned lane_blocks, const unsigned n_rows, const int unroll)
{
    const unsigned tid = threadIdx.x, lane = tid & 31u;
    const bool by_warp = P.mode == 1;
    const int lane_var = P.lane_var;
    const int share = (int)blockIdx.y;
    const float *__restrict__ src0 = ptrs.in[P.loads[0].ptr];
    const float *__restrict__ src1 = P.n_loads > 1 ? ptrs.in[P.loads[1].ptr] : src0;
    const float *__restrict__ src2 = P.n_loads > 2 ? ptrs.in[P.loads[2].ptr] : src0;
    const float *__restrict__ src3 = P.n_loads > 3 ? ptrs.in[P.loads[3].ptr] : src0;
    const int n_loads = P.n_loads;
    const float *const srcs[4] = {src0, src1, src2, src3};
    const int sq[4] = {P.loads[0].sq, P.loads[1].sq, P.loads[2].sq, P.loads[3].sq};
    for (unsigned item = blockIdx.x; item < n_items; item += gridDim.x) {
        // the output of this thread (mode 0) or warp (mode 1)
        unsigned row, lane0;
        bool exists;
        if (by_warp) {
            const unsigned w = item * 8u + (tid >> 5);            // flat output index
            row = w / (unsigned)P.outer_ext[lane_var]; lane0 = w - row * (unsigned)P.outer_ext[lane_var];
            exists = row < n_rows;
        } else {
            const unsigned rows_per_block = 256u / cols, tc = tid % cols, tr = tid / cols;
            const unsigned lb = item % lane_blocks, rb = item / lane_blocks;
            row = rb * rows_per_block + tr; lane0 = lb * cols + tc;
            exists = row < n_rows && lane0 < (unsigned)P.outer_ext[lane_var];
        }
        if (!exists) continue;
        int var[V];
        unsigned rem = row;
#pragma unroll
        for (int v = V - 1; v >= 0; --v) {
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
        bool live = true;
        for (int r = 0; r < P.n_guards; ++r) if (row_num(P.guards[r], var, 0) > 0) live = false;
        float acc = 0.f;
        if (live) {
            // offsets at z = 0
            int b0 = P.loads[0].base, b1 = P.loads[1].base, b2 = P.loads[2].base, b3 = P.loads[3].base;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                b0 += P.loads[0].coef[v] * var[v]; b1 += P.loads[1].coef[v] * var[v];
                b2 += P.loads[2].coef[v] * var[v]; b3 += P.loads[3].coef[v] * var[v];
            }
            int lo0, hi0;
            range(P, 0, var, 0, lo0, hi0);
            if (P.n_share[0] > 1) {
                // pieces of the loop's box, counted from the one this output's range starts in: every share is short
                const int s0 = P.n_share[1] == 1 ? share : share / P.n_share[1];
                const int a = P.zbox_lo[0] + ((((lo0 - P.zbox_lo[0]) >> P.chunk_shift[0]) + s0) << P.chunk_shift[0]);
                lo0 = max(lo0, a); hi0 = min(hi0, a + (1 << P.chunk_shift[0]) - 1);
            }
            const bool two = P.n_loops == 2;
            const int step_in = by_warp ? 32 : 1, first_in = by_warp ? (int)lane : 0;
            // the innermost loop advances every offset by its own step
            const int l_in = two ? 1 : 0;
            const int d0 = P.loads[0].cz[l_in] * step_in, d1 = P.loads[1].cz[l_in] * step_in;
            const int d2 = P.loads[2].cz[l_in] * step_in, d3 = P.loads[3].cz[l_in] * step_in;
            for (int z0 = lo0; z0 <= (two ? hi0 : lo0); ++z0) {
                int lo = lo0, hi = hi0;
                int o0 = b0, o1 = b1, o2 = b2, o3 = b3;
                if (two) {
                    range(P, 1, var, z0, lo, hi);
                    if (P.n_share[1] > 1) {
                        const int a = P.zbox_lo[1] + ((((lo - P.zbox_lo[1]) >> P.chunk_shift[1]) + share % P.n_share[1]) << P.chunk_shift[1]);
                        lo = max(lo, a); hi = min(hi, a + (1 << P.chunk_shift[1]) - 1);
                    }
                    o0 += P.loads[0].cz[0] * z0; o1 += P.loads[1].cz[0] * z0; o2 += P.loads[2].cz[0] * z0; o3 += P.loads[3].cz[0] * z0;
                }
                const int zs = lo + first_in;
                o0 += P.loads[0].cz[l_in] * zs; o1 += P.loads[1].cz[l_in] * zs; o2 += P.loads[2].cz[l_in] * zs; o3 += P.loads[3].cz[l_in] * zs;
                int o[4] = {o0, o1, o2, o3};
                const int d[4] = {d0, d1, d2, d3};
                float part;
#define TAD_WALK(NL) (unroll == 2 ? walk<NL, 2, STREAM>(srcs, sq, o, d, zs, hi, step_in) : unroll == 4 ? walk<NL, 4, STREAM>(srcs, sq, o, d, zs, hi, step_in) : walk<NL, 8, STREAM>(srcs, sq, o, d, zs, hi, step_in))
                if (n_loads == 1) part = TAD_WALK(1);
                else if (n_loads == 2) part = TAD_WALK(2);
                else if (n_loads == 3) part = TAD_WALK(3);
                else part = TAD_WALK(4);
#undef TAD_WALK
                acc += part;
            }
        }
        if (by_warp) {
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
            if (lane != 0) continue;
        }
        // the factor outside the sums
        float sc = P.cscale * P.cterm;
        for (int q = 0; q < P.n_scale; ++q) {
            int o = P.scale[q].base;
#pragma unroll
            for (int v = 0; v < V; ++v) o += P.scale[q].coef[v] * var[v];
            if (live) sc *= __ldg(ptrs.in[P.scale[q].ptr] + (unsigned)o);
        }
        const float result = live ? acc * sc : 0.f;
        if (P.zsplit > 1) {
            unsigned cell = 0;
#pragma unroll
            for (int v = 0; v < V; ++v) if (v < P.n_outer) cell += (unsigned)P.part_coef[v] * (unsigned)(var[v] - P.outer_lo[v]);
            ptrs.part[(size_t)share * (unsigned)P.part_limit + cell] = result;
            if (P.live_plane && share == 0) ptrs.part[(size_t)P.zsplit * (unsigned)P.part_limit + cell] = live ? 1.f : 0.f;
        } else {
            int o = P.out_base;
#pragma unroll
            for (int v = 0; v < V; ++v) o += P.out_coef[v] * var[v];
            if (P.accumulate) { if (live) ptrs.out[(unsigned)o] += result; }
            else ptrs.out[(unsigned)o] = result;
        }
    }
}

}  // namespace

cudaError_t tad_launch_line(const TadlProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream)
{
    const unsigned lane_ext = (unsigned)P.outer_ext[P.lane_var];
    unsigned long long rows = 1;
    for (int v = 0; v < P.n_outer; ++v) if (v != P.lane_var) rows *= (unsigned long long)P.outer_ext[v];
    if (lane_ext == 0 || rows == 0) return cudaSuccess;
    unsigned cols = 1, lane_blocks = 1;
    unsigned long long items;
    if (P.mode == 1) items = (rows * lane_ext + 7) / 8;                 // eight warps, eight outputs per block
    else {
        while (cols < 256u && cols < lane_ext) cols *= 2u;
        lane_blocks = (lane_ext + cols - 1u) / cols;
        items = ((rows + 256u / cols - 1) / (256u / cols)) * lane_blocks;
    }
    if (items >= (1ull << 31) || rows >= (1ull << 31)) return cudaErrorInvalidValue;
    const unsigned gx = (unsigned)std::min<unsigned long long>(items, (unsigned long long)sms * 32ull);
    dim3 grid(gx, (unsigned)std::max(1, P.zsplit), 1u);
    if (P.stream) tad_line_kernel<true><<<grid, 256, 0, stream>>>(P, ptrs, (unsigned)items, cols, lane_blocks, (unsigned)rows, P.unroll);
    else tad_line_kernel<false><<<grid, 256, 0, stream>>>(P, ptrs, (unsigned)items, cols, lane_blocks, (unsigned)rows, P.unroll);
    return cudaGetLastError();
}

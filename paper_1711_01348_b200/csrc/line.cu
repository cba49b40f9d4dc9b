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

__global__ void __launch_bounds__(256)
tad_line_kernel(const __grid_constant__ TadlProgram P, const __grid_constant__ TadpPointers ptrs, const unsigned n_items,
                const unsigned cols, const unsigned lane_blocks, const unsigned n_rows)
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
            if (P.zsplit > 1 && hi0 >= lo0) {
                // share s of the range: [lo + len * s / S, lo + len * (s + 1) / S)
                const long long len = (long long)hi0 - lo0 + 1;
                const int a = lo0 + (int)(len * share / P.zsplit), b = lo0 + (int)(len * (share + 1) / P.zsplit) - 1;
                lo0 = a; hi0 = b;
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
                    o0 += P.loads[0].cz[0] * z0; o1 += P.loads[1].cz[0] * z0; o2 += P.loads[2].cz[0] * z0; o3 += P.loads[3].cz[0] * z0;
                }
                const int zs = lo + first_in;
                o0 += P.loads[0].cz[l_in] * zs; o1 += P.loads[1].cz[l_in] * zs; o2 += P.loads[2].cz[l_in] * zs; o3 += P.loads[3].cz[l_in] * zs;
                float s0 = 0.f, s1 = 0.f;
                int z = zs;
                if (n_loads == 1) {
                    for (; z + step_in <= hi; z += 2 * step_in) { s0 += __ldg(src0 + (unsigned)o0); s1 += __ldg(src0 + (unsigned)(o0 + d0)); o0 += 2 * d0; }
                    if (z <= hi) s0 += __ldg(src0 + (unsigned)o0);
                } else if (n_loads == 2) {
                    for (; z + step_in <= hi; z += 2 * step_in) {
                        const float x0 = __ldg(src0 + (unsigned)o0), y0 = __ldg(src1 + (unsigned)o1);
                        const float x1 = __ldg(src0 + (unsigned)(o0 + d0)), y1 = __ldg(src1 + (unsigned)(o1 + d1));
                        s0 = fmaf(x0, y0, s0); s1 = fmaf(x1, y1, s1);
                        o0 += 2 * d0; o1 += 2 * d1;
                    }
                    if (z <= hi) s0 = fmaf(__ldg(src0 + (unsigned)o0), __ldg(src1 + (unsigned)o1), s0);
                } else if (n_loads == 3) {
                    for (; z + step_in <= hi; z += 2 * step_in) {
                        const float x0 = __ldg(src0 + (unsigned)o0), y0 = __ldg(src1 + (unsigned)o1), w0 = __ldg(src2 + (unsigned)o2);
                        const float x1 = __ldg(src0 + (unsigned)(o0 + d0)), y1 = __ldg(src1 + (unsigned)(o1 + d1)), w1 = __ldg(src2 + (unsigned)(o2 + d2));
                        s0 = fmaf(x0 * y0, w0, s0); s1 = fmaf(x1 * y1, w1, s1);
                        o0 += 2 * d0; o1 += 2 * d1; o2 += 2 * d2;
                    }
                    if (z <= hi) s0 = fmaf(__ldg(src0 + (unsigned)o0) * __ldg(src1 + (unsigned)o1), __ldg(src2 + (unsigned)o2), s0);
                } else {
                    for (; z <= hi; z += step_in) {
                        s0 = fmaf(__ldg(src0 + (unsigned)o0) * __ldg(src1 + (unsigned)o1), __ldg(src2 + (unsigned)o2) * __ldg(src3 + (unsigned)o3), s0);
                        o0 += d0; o1 += d1; o2 += d2; o3 += d3;
                    }
                }
                acc += s0 + s1;
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
    tad_line_kernel<<<grid, 256, 0, stream>>>(P, ptrs, (unsigned)items, cols, lane_blocks, (unsigned)rows);
    return cudaGetLastError();
}

// The interpreter kernel for one vector shape (TAD_TA x TAD_UB, given on the command line) and its launcher.
#include <cuda_runtime.h>

#include <algorithm>

#include "vm.cuh"

#ifndef TAD_TA
#error "compile with -DTAD_TA=<n> -DTAD_UB=<n>"
#endif

namespace {

using namespace tadvm;

// One warp per work item, grid-stride over the items.  A work item fixes every outer variable
// except the lane variable A, which the warp covers 32 * TA values at a time, and the element
// variable B when that is an outer variable, which it covers UB values at a time.
template <int TA, int UB, bool DEBUG, bool REL>
__global__ void __launch_bounds__(VmCfg<TA, UB>::WARPS * 32, (TA * UB >= 32 ? 3 : 2))
tad_vm_kernel(const __grid_constant__ TadpProgram P, const __grid_constant__ TadpPointers ptrs, unsigned n_items)
{
    constexpr int E = TA * UB;
    const unsigned lane = threadIdx.x & 31u;
    const unsigned warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const unsigned n_warps = (gridDim.x * blockDim.x) >> 5;
    const int lane_var = P.lane_var;
    const int unroll_var = P.unroll_var;
    const bool lane_outer = lane_var < P.n_outer;
    const bool unroll_outer = UB > 1 && P.unroll_kind == 1;
    Vm<TA, UB> m;
    const unsigned zsplit = P.zsplit > 1 ? (unsigned)P.zsplit : 1u;
    for (unsigned witem = warp; witem < n_items; witem += n_warps) {
        // warps witem = item * zsplit + s share the outputs of `item`
        const unsigned item = witem / zsplit;
        const int split = (int)(witem % zsplit);
        // decode the outer variables (last one fastest)
        unsigned rem = item;
#pragma unroll
        for (int k = 0; k < TADP_MAX_VARS; ++k) m.var[k] = 0;
        unsigned first_a = 0, ext_a = 0xffffffffu, first_b = 0, ext_b = 0xffffffffu;
#pragma unroll
        for (int v = TADP_MAX_VARS - 1; v >= 0; --v) {
            if (v < P.n_outer) {
                const unsigned ext = (unsigned)P.outer_ext[v];
                if (v == lane_var) {
                    const unsigned chunks = (ext + 32u * TA - 1u) / (32u * TA);
                    const unsigned c = rem % chunks; rem /= chunks;
                    first_a = c * 32u * TA + lane; ext_a = ext;
                    m.var[v] = P.outer_lo[v] + (int)first_a;
                } else if (unroll_outer && v == unroll_var) {
                    const unsigned chunks = (ext + UB - 1u) / UB;
                    const unsigned c = rem % chunks; rem /= chunks;
                    first_b = c * UB; ext_b = ext;
                    m.var[v] = P.outer_lo[v] + (int)first_b;
                } else {
                    const unsigned c = rem % ext; rem /= ext;
                    m.var[v] = P.outer_lo[v] + (int)c;
                }
            }
        }
        unsigned mask0 = 0;
#pragma unroll
        for (int e = 0; e < E; ++e)
            if (first_a + 32u * (e / UB) < ext_a && first_b + (unsigned)(e % UB) < ext_b) mask0 |= 1u << e;
        const unsigned in_range = mask0;
        // guards: rows over the outer variables that must be <= 0 for Gamma to be non-empty
        for (int r = 0; r < P.n_guards; ++r) {
            const TadpRow &R = P.rows[P.guard0 + r];
            const int nmr = row_num(R, m.var);
            const int sa = lane_outer ? R.coef[lane_var] * 32 : 0;
            const int sb = unroll_outer ? R.coef[unroll_var] : 0;
#pragma unroll
            for (int e = 0; e < E; ++e) if (nmr + (e / UB) * sa + (e % UB) * sb > 0) mask0 &= ~(1u << e);
        }
        unsigned live = 0;
        run_item<TA, UB, DEBUG, REL>(P, ptrs, m, mask0, split, live);

        // ---- output: distinct elements along t when A is an outer variable, along u when B is ----
        const int n_u = unroll_outer ? UB : 1;
        unsigned off = (unsigned)P.out_base;
#pragma unroll
        for (int k = 0; k < TADP_MAX_VARS; ++k) if (k < P.n_outer) off += (unsigned)P.out_coef[k] * (unsigned)m.var[k];
        const unsigned step_a = lane_outer ? (unsigned)P.out_coef[lane_var] * 32u : 0u;
        const unsigned step_b = unroll_outer ? (unsigned)P.out_coef[unroll_var] : 0u;
        if (zsplit > 1) {
            // this warp's share of the sums goes to its plane of partial sums, indexed compactly
            // by the outer variables; a second launch adds the planes up in order
            unsigned cidx = 0;
#pragma unroll
            for (int k = 0; k < TADP_MAX_VARS; ++k) if (k < P.n_outer) cidx += (unsigned)P.part_coef[k] * (unsigned)(m.var[k] - P.outer_lo[k]);
            const unsigned cstep_a = lane_outer ? (unsigned)P.part_coef[lane_var] * 32u : 0u;
            const unsigned cstep_b = unroll_outer ? (unsigned)P.part_coef[unroll_var] : 0u;
            float *plane = ptrs.part + (size_t)split * (unsigned)P.part_limit;
            float *flags = ptrs.part + (size_t)zsplit * (unsigned)P.part_limit;
            if (lane_outer) {
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if ((e % UB) >= n_u || !((in_range >> e) & 1u)) continue;
                    const unsigned c = cidx + (unsigned)(e / UB) * cstep_a + (unsigned)(e % UB) * cstep_b;
                    plane[c] = m.acc[e];
                    if ((live >> e) & 1u) flags[c] = 1.f;
                }
            } else {
#pragma unroll
                for (int u = 0; u < UB; ++u) {
                    if (u >= n_u) continue;
                    float total = 0.f;
                    unsigned lv = 0;
#pragma unroll
                    for (int t = 0; t < TA; ++t) { total += m.acc[t * UB + u]; lv |= (live >> (t * UB + u)) & 1u; }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
                    const unsigned any_live = __ballot_sync(0xffffffffu, lv != 0);
                    if (lane == 0 && first_b + (unsigned)u < ext_b) {
                        const unsigned c = cidx + (unsigned)u * cstep_b;
                        plane[c] = total;
                        if (any_live) flags[c] = 1.f;
                    }
                }
            }
            continue;
        }
        float *dst = ptrs.out;
        const bool accumulate = P.accumulate != 0;
        const bool only_live = P.write_only_live != 0;
        constexpr unsigned FULL_MASK = E >= 32 ? 0xffffffffu : ((1u << E) - 1u);
        if (!DEBUG && lane_outer && n_u == UB && in_range == FULL_MASK && !only_live) {
            // a full tile of outputs: no test per element
            if (accumulate) {
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const unsigned idx = off + (unsigned)(e / UB) * step_a + (unsigned)(e % UB) * step_b;
                    dst[idx] += m.acc[e];
                }
            } else {
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const unsigned idx = off + (unsigned)(e / UB) * step_a + (unsigned)(e % UB) * step_b;
                    dst[idx] = m.acc[e];
                }
            }
        } else if (lane_outer) {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                if ((e % UB) >= n_u) continue;
                if (!((in_range >> e) & 1u)) continue;
                if (only_live && !((live >> e) & 1u)) continue;
                const unsigned idx = off + (unsigned)(e / UB) * step_a + (unsigned)(e % UB) * step_b;
                if (DEBUG && idx >= (unsigned)P.out_limit) { if (ptrs.debug) atomicCAS(ptrs.debug, 0, 0x20000); continue; }
                dst[idx] = accumulate ? dst[idx] + m.acc[e] : m.acc[e];
            }
        } else {
            // the lane variable is a kernel coordinate: fixed-order tree reduction over t and the lanes
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                if (u >= n_u) continue;
                float total = 0.f;
                unsigned lv = 0;
#pragma unroll
                for (int t = 0; t < TA; ++t) { total += m.acc[t * UB + u]; lv |= (live >> (t * UB + u)) & 1u; }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
                const unsigned any_live = __ballot_sync(0xffffffffu, lv != 0);
                const bool inside = first_b + (unsigned)u < ext_b;
                if (lane == 0 && inside && !(only_live && !any_live)) {
                    const unsigned idx = off + (unsigned)u * step_b;
                    if (DEBUG && idx >= (unsigned)P.out_limit) { if (ptrs.debug) atomicCAS(ptrs.debug, 0, 0x20000); }
                    else dst[idx] = accumulate ? dst[idx] + total : total;
                }
            }
        }
    }
}

}  // namespace

#define TAD_CAT3(a, b, c, d) a##b##c##d
#if TAD_RICH_BUILD
#define TAD_CAT4(a, b, c, d, e) a##b##c##d##e
#define TAD_LAUNCH_NAME(TA, UB) TAD_CAT4(tad_launch_vm_, TA, _, UB, _rich)
#else
#define TAD_LAUNCH_NAME(TA, UB) TAD_CAT3(tad_launch_vm_, TA, _, UB)
#endif

// Builds per shape: plain, with the relative-loop support (no element variable) and, for narrow
// shapes, with bounds checks.  False when the shape has no build for what the program asks: nothing was launched.
bool TAD_LAUNCH_NAME(TAD_TA, TAD_UB)(const TadpProgram &prog, const TadpPointers &ptrs, bool debug, unsigned items, unsigned sms, cudaStream_t stream)
{
    constexpr int TA = TAD_TA, UB = TAD_UB;
    constexpr unsigned WPB = VmCfg<TA, UB>::WARPS;
    // one warp per work item, grid-stride; at most 128 warps' worth of blocks per SM
    const unsigned blocks = std::min((items + WPB - 1) / WPB, sms * (128u / WPB));
    if (debug) {
        if constexpr (TA <= 4 && UB == 1) tad_vm_kernel<TA, UB, true, true><<<blocks, WPB * 32, 0, stream>>>(prog, ptrs, items);
        else return false;
    } else if (prog.rel_var >= 0) {
        if constexpr (UB == 1) tad_vm_kernel<TA, UB, false, true><<<blocks, WPB * 32, 0, stream>>>(prog, ptrs, items);
        else return false;
    } else tad_vm_kernel<TA, UB, false, false><<<blocks, WPB * 32, 0, stream>>>(prog, ptrs, items);
    return true;
}

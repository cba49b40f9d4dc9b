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


// ---------------------------------------------------------------------------------------------------------
// Products of loads.  Most element-wise kernels that remain after the function tables are
//     out = c * L_1^e1 * L_2^e2 * ...        (e in 1..3),
// and at one multiplication per load the index arithmetic of the general program dominates.  Here a thread
// owns four outputs of a row and walks a run of consecutive rows along another outer variable, so the
// variables are decoded once per run and every offset advances by a constant per row.  Two layouts:
//   vector:      the four outputs are consecutive; every load that moves along the row is a 128-bit load
//                (forward, or reversed for offsets that step by -1), which the host has proven aligned in every row;
//   interleaved: output j of a thread lies j * (threads per row) further, so that plain loads of neighbouring
//                threads fall into the same lines whatever the load's step.
// Loads that do not change from row to row are read once per run, loads that do not move along the row once per row.
// ---------------------------------------------------------------------------------------------------------
enum ProdKind : int { PK_HOIST = 0, PK_BCAST, PK_FWD, PK_REV, PK_GEN };

struct ProdLoad { int32_t load, kind, exp; };
struct ProdPlan {
    int32_t n_loads, n_moving, row_var, run, vec;      // run: rows per thread along row_var (row_var < 0: single rows); moving loads first
    float c;
    ProdLoad ld[4];
};

__device__ __forceinline__ float powe(float v, int e) { return e == 1 ? v : e == 2 ? v * v : v * v * v; }

template <bool VEC, int M>
__global__ void __launch_bounds__(256, 3)
tad_prod_kernel(const __grid_constant__ TadeProgram P, const __grid_constant__ ProdPlan Q, const __grid_constant__ TadpPointers ptrs,
                const unsigned n_items, const unsigned cols, const unsigned lane_blocks, const unsigned n_runs, const unsigned runs_per_line)
{
    const unsigned tid = threadIdx.x;
    const unsigned rows_per_block = 256u / cols;
    const unsigned tc = tid % cols, tr = tid / cols;
    const int lane_var = P.lane_var, row_var = Q.row_var;
    const unsigned lane_ext = (unsigned)P.outer_ext[lane_var];
    const unsigned es = VEC ? 1u : cols;                       // distance between two outputs of a thread
    float *__restrict__ out = ptrs.out;
    for (unsigned item = blockIdx.x; item < n_items; item += gridDim.x) {
        const unsigned lb = item % lane_blocks, rb = item / lane_blocks;
        const unsigned run = rb * rows_per_block + tr;
        const unsigned lane0 = lb * cols * 4u + (VEC ? tc * 4u : tc);
        if (run >= n_runs || lane0 >= lane_ext) continue;
        int live;                                              // outputs of this thread inside the row
        if (VEC) live = (int)min(4u, lane_ext - lane0);
        else live = (int)min(4u, (lane_ext - lane0 + cols - 1u) / cols);
        // the run: its position along row_var, then the other outer variables
        const unsigned piece = run % runs_per_line;
        unsigned rem = run / runs_per_line;
        int var[TADP_MAX_VARS];
#pragma unroll
        for (int v = TADP_MAX_VARS - 1; v >= 0; --v) {
            var[v] = 0;
            if (v < P.n_outer) {
                if (v == lane_var) var[v] = P.outer_lo[v] + (int)lane0;
                else if (v == row_var) var[v] = P.outer_lo[v] + (int)(piece * (unsigned)Q.run);
                else {
                    const unsigned q = (unsigned)(((unsigned long long)rem * (unsigned)P.div_mul[v]) >> P.div_shift[v]);
                    var[v] = P.outer_lo[v] + (int)(rem - q * (unsigned)P.outer_ext[v]);
                    rem = q;
                }
            }
        }
        const int n_rows = row_var < 0 ? 1 : min(Q.run, P.outer_ext[row_var] - (int)(piece * (unsigned)Q.run));
        // loads that stay put from row to row are multiplied into one factor per output (with the constant); the
        // others ("moving", Q.n_moving of them, first in Q.ld) keep an offset that advances by a constant per row
        float held[4] = {Q.c, Q.c, Q.c, Q.c};
        int off[3] = {0, 0, 0}, step[3] = {0, 0, 0}, adv[3] = {0, 0, 0}, kinds[3] = {0, 0, 0}, exps[3] = {1, 1, 1};
        const float *__restrict__ srcs[3] = {nullptr, nullptr, nullptr};
        constexpr int n_moving = M;
        unsigned widths = 0x111u;                              // four bits per moving load: values per vector load in this run
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            if (l >= Q.n_loads) continue;
            const TadpLoad &L = P.loads[Q.ld[l].load];
            int o = L.base;
#pragma unroll
            for (int v = 0; v < TADP_MAX_VARS; ++v) o += L.coef[v] * var[v];
            const int st = L.coef[lane_var] * (int)es;
            if (l >= M) {
                const float *__restrict__ src = ptrs.in[L.ptr];
#pragma unroll
                for (int j = 0; j < 4; ++j) if (j < live) held[j] *= powe(__ldg(src + (unsigned)(o + j * st)), Q.ld[l].exp);
            } else if (l < 3) {
                off[l] = o; step[l] = st; adv[l] = L.coef[row_var];
                kinds[l] = Q.ld[l].kind; exps[l] = Q.ld[l].exp; srcs[l] = ptrs.in[L.ptr];
                if (VEC && live == 4 && (Q.ld[l].kind == PK_FWD || Q.ld[l].kind == PK_REV)) {
                    const unsigned first = (unsigned)(Q.ld[l].kind == PK_FWD ? o : o - 3);
                    widths += ((first & 3u) == 0 ? 3u : (first & 1u) == 0 ? 1u : 0u) << (4 * l);
                }
            }
        }
        int oo = P.out_base;
#pragma unroll
        for (int v = 0; v < TADP_MAX_VARS; ++v) oo += P.out_coef[v] * var[v];
        const int ostep = P.out_coef[lane_var] * (int)es, oadv = row_var < 0 ? 0 : P.out_coef[row_var];
        // the product of one row (offsets advance to the next row)
        auto row = [&](float (&p)[4]) {
#pragma unroll
            for (int j = 0; j < 4; ++j) p[j] = held[j];
#pragma unroll
            for (int l = 0; l < M; ++l) {
                const int kind = kinds[l];
                const unsigned w = (widths >> (4 * l)) & 15u;
                const float *__restrict__ src = srcs[l];
                float v4[4];
                if (kind == PK_BCAST) {
                    const float s = __ldg(src + (unsigned)off[l]);
                    v4[0] = v4[1] = v4[2] = v4[3] = s;
                } else if (VEC && w == 4u) {
                    if (kind == PK_FWD) {
                        const float4 q = __ldg(reinterpret_cast<const float4 *>(src + (unsigned)off[l]));
                        v4[0] = q.x; v4[1] = q.y; v4[2] = q.z; v4[3] = q.w;
                    } else {
                        const float4 q = __ldg(reinterpret_cast<const float4 *>(src + (unsigned)(off[l] - 3)));
                        v4[0] = q.w; v4[1] = q.z; v4[2] = q.y; v4[3] = q.x;
                    }
                } else if (VEC && w == 2u) {
                    if (kind == PK_FWD) {
                        const float2 q0 = __ldg(reinterpret_cast<const float2 *>(src + (unsigned)off[l]));
                        const float2 q1 = __ldg(reinterpret_cast<const float2 *>(src + (unsigned)(off[l] + 2)));
                        v4[0] = q0.x; v4[1] = q0.y; v4[2] = q1.x; v4[3] = q1.y;
                    } else {
                        const float2 q0 = __ldg(reinterpret_cast<const float2 *>(src + (unsigned)(off[l] - 1)));
                        const float2 q1 = __ldg(reinterpret_cast<const float2 *>(src + (unsigned)(off[l] - 3)));
                        v4[0] = q0.y; v4[1] = q0.x; v4[2] = q1.y; v4[3] = q1.x;
                    }
                } else if (live == 4) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) v4[j] = __ldg(src + (unsigned)(off[l] + j * step[l]));
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) v4[j] = j < live ? __ldg(src + (unsigned)(off[l] + j * step[l])) : 0.f;
                }
                if (exps[l] != 1) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) v4[j] = powe(v4[j], exps[l]);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) p[j] *= v4[j];
                off[l] += adv[l];
            }
        };
        auto store = [&](const float (&p)[4]) {
            if (VEC && live == 4) {
                float4 *dst = reinterpret_cast<float4 *>(out + (unsigned)oo);
                float4 q = make_float4(p[0], p[1], p[2], p[3]);
                if (P.accumulate) { const float4 o = *dst; q.x += o.x; q.y += o.y; q.z += o.z; q.w += o.w; }
                *dst = q;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < live) { const unsigned o = (unsigned)(oo + j * ostep); out[o] = P.accumulate ? out[o] + p[j] : p[j]; }
            }
            oo += oadv;
        };
        // two rows in flight: the loads of the second are issued before the first is multiplied and stored
        int r = 0;
        for (; r + 2 <= n_rows; r += 2) {
            float p0[4], p1[4];
            row(p0); row(p1);
            store(p0); store(p1);
        }
        if (r < n_rows) { float p0[4]; row(p0); store(p0); }
    }
}

// c * product of powers of loads, read off the accumulator program; false when the program is anything else
bool product_form(const TadeProgram &P, ProdPlan &Q)
{
    struct Group { float c; int exp[TADE_MAX_LOADS]; bool any; };
    Group x{}, y{};
    bool have_x = false, have_y = false;
    auto raise = [](Group &g, int k) {
        for (int l = 0; l < TADE_MAX_LOADS; ++l) { g.exp[l] *= k; if (g.exp[l] > 3) return false; }
        g.c = k == 2 ? g.c * g.c : g.c * g.c * g.c;
        return true;
    };
    for (int s = 0; s < P.n_steps; ++s) {
        const TadeStep &st = P.steps[s];
        switch (st.op) {
        case E_LD:
            if (st.a < 0 || st.a >= TADE_MAX_LOADS) return false;
            if (st.b == 0) { x = Group{}; x.c = 1.f; x.exp[st.a] = 1; have_x = true; }
            else if (st.b == 2 && have_x) { if (++x.exp[st.a] > 3) return false; }
            else return false;
            break;
        case E_PUSH: if (!have_x || have_y) return false; y = x; have_y = true; have_x = false; break;
        case E_NEG: if (!have_x) return false; x.c = -x.c; break;
        case E_MULC: if (!have_x) return false; x.c *= st.imm; break;
        case E_SQR: if (!have_x || !raise(x, 2)) return false; break;
        case E_CUBE: if (!have_x || !raise(x, 3)) return false; break;
        case E_MULY:
            if (!have_x || !have_y) return false;
            x.c *= y.c;
            for (int l = 0; l < TADE_MAX_LOADS; ++l) { x.exp[l] += y.exp[l]; if (x.exp[l] > 3) return false; }
            have_y = false;
            break;
        default: return false;
        }
    }
    if (!have_x || have_y) return false;
    Q = ProdPlan{};
    Q.c = x.c;
    for (int l = 0; l < TADE_MAX_LOADS; ++l)
        if (x.exp[l] > 0) {
            if (Q.n_loads == 4 || l >= P.n_loads) return false;
            Q.ld[Q.n_loads].load = l; Q.ld[Q.n_loads].exp = x.exp[l]; ++Q.n_loads;
        }
    return Q.n_loads > 0;
}

// layout and load kinds of a product program; the row variable is the innermost outer variable besides the lane variable
bool plan_product(const TadeProgram &P, const TadpPointers &ptrs, unsigned sms, ProdPlan &Q)
{
    const int lane = P.lane_var;
    Q.row_var = -1;
    for (int v = P.n_outer - 1; v >= 0; --v) if (v != lane && P.outer_ext[v] > 1) { Q.row_var = v; break; }
    double elems = 1;
    for (int v = 0; v < P.n_outer; ++v) elems *= (double)P.outer_ext[v];
    // rows per thread: as many as leave every SM a few thousand threads
    int run = 1;
    while (run < 32 && elems / (4.0 * run * 2) >= (double)sms * 2048.0) run *= 2;
    Q.run = Q.row_var < 0 ? 1 : std::min(run, P.outer_ext[Q.row_var]);
    // the output is stored in 128-bit pieces when its first element of every row is a multiple of four; a load needs
    // only a row step that is one (the width of its vector loads is settled per run)
    auto aligned = [&](const int32_t *coef, int64_t base) {
        int64_t o = base;
        for (int v = 0; v < P.n_outer; ++v) { o += (int64_t)coef[v] * P.outer_lo[v]; if (v != lane && coef[v] % 4 != 0) return false; }
        return o % 4 == 0;
    };
    bool vec = P.out_coef[lane] == 1 && aligned(P.out_coef, P.out_base) && (reinterpret_cast<uintptr_t>(ptrs.out) & 15u) == 0;
    for (int i = 0; i < Q.n_loads; ++i) {
        const TadpLoad &L = P.loads[Q.ld[i].load];
        const int step = L.coef[lane], adv = Q.row_var < 0 ? 0 : L.coef[Q.row_var];
        const bool base16 = (reinterpret_cast<uintptr_t>(ptrs.in[L.ptr]) & 15u) == 0;
        int kind = PK_GEN;
        if (adv == 0 || Q.run == 1) kind = PK_HOIST;
        else if (step == 0) kind = PK_BCAST;
        else if (step == 1 && base16 && adv % 4 == 0) kind = PK_FWD;
        else if (step == -1 && base16 && adv % 4 == 0) kind = PK_REV;
        if (kind == PK_GEN) vec = false;
        Q.ld[i].kind = kind;
    }
    // moving loads first
    std::stable_sort(Q.ld, Q.ld + Q.n_loads, [](const ProdLoad &a, const ProdLoad &b) { return (a.kind != PK_HOIST) > (b.kind != PK_HOIST); });
    Q.n_moving = 0;
    for (int i = 0; i < Q.n_loads; ++i) Q.n_moving += Q.ld[i].kind != PK_HOIST;
    Q.vec = vec ? 1 : 0;
    return Q.n_moving <= 3;
}

}  // namespace

cudaError_t tad_launch_ew(const TadeProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream)
{
    const unsigned lane_ext = (unsigned)P.outer_ext[P.lane_var];
    unsigned long long rows = 1;
    for (int v = 0; v < P.n_outer; ++v) if (v != P.lane_var) rows *= (unsigned long long)P.outer_ext[v];
    if (lane_ext == 0 || rows == 0) return cudaSuccess;
    ProdPlan Q;
    if (product_form(P, Q) && plan_product(P, ptrs, sms, Q)) {
        unsigned pc = 1;
        while (pc < 256u && pc * 4u < lane_ext) pc *= 2u;
        if (!Q.vec && pc < 32u) pc = 32u;                      // interleaved outputs: a warp covers a run of 32 columns
        const unsigned per_block = 256u / pc;
        const unsigned lblocks = (lane_ext + pc * 4u - 1u) / (pc * 4u);
        const unsigned long long row_ext = Q.row_var < 0 ? 1ull : (unsigned long long)P.outer_ext[Q.row_var];
        const unsigned long long per_line = (row_ext + Q.run - 1) / Q.run;
        const unsigned long long runs = rows / row_ext * per_line;
        const unsigned long long its = ((runs + per_block - 1) / per_block) * lblocks;
        if (its >= (1ull << 32) || runs >= (1ull << 31)) return cudaErrorInvalidValue;
        const unsigned g = (unsigned)std::min<unsigned long long>(its, (unsigned long long)sms * 32ull);
#define TAD_PROD_LAUNCH(V, MM) tad_prod_kernel<V, MM><<<g, 256, 0, stream>>>(P, Q, ptrs, (unsigned)its, pc, lblocks, (unsigned)runs, (unsigned)per_line)
        switch ((Q.vec ? 4 : 0) + Q.n_moving) {
        case 0: TAD_PROD_LAUNCH(false, 0); break;
        case 1: TAD_PROD_LAUNCH(false, 1); break;
        case 2: TAD_PROD_LAUNCH(false, 2); break;
        case 3: TAD_PROD_LAUNCH(false, 3); break;
        case 4: TAD_PROD_LAUNCH(true, 0); break;
        case 5: TAD_PROD_LAUNCH(true, 1); break;
        case 6: TAD_PROD_LAUNCH(true, 2); break;
        default: TAD_PROD_LAUNCH(true, 3); break;
        }
#undef TAD_PROD_LAUNCH
        return cudaGetLastError();
    }
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

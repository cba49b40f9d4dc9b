// Warp-uniform bytecode interpreter.
//
// One warp runs one work item at a time: the outer variables of the item are decoded from the
// item number, the lane variable is spread over the 32 lanes and over T vector elements per
// lane (element t of lane l has coordinate base + l + 32 t, so that every vector element of a
// load is one fully coalesced warp transaction).  All control flow (program counter, loop
// trip counts) is uniform across the warp; per-element validity is a T-bit activity mask.
//
// The operand stack is a register array indexed only by compile-time constants: the host
// encodes the stack depth (or, for loop control, the loop variable) into the handler number
// of every instruction, so each handler names its registers statically and nothing of the
// stack spills to local memory.  exp, sin, cos and tanh are evaluated inline, a word's values side
// by side; the other elementary functions are out-of-line calls so that the handler code stays
// small.  Innermost loops whose body is a short chain of loads and arithmetic run inside one
// word (P_XLOOP); in the 32-value shapes that word runs products of two loads in loops of their own.
#pragma once
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "program.h"

namespace tadvm {

constexpr int STACK = TADP_MAX_DEPTH - 1;   // usable depth (handlers are encoded for depth 0..7)

__device__ __forceinline__ int floor_div_i(int a, int b) { int q = a / b; return (a % b != 0 && a < 0) ? q - 1 : q; }
__device__ __forceinline__ int ceil_div_i(int a, int b) { int q = a / b; return (a % b != 0 && a > 0) ? q + 1 : q; }

// The handlers of one operation differ only in which registers they touch.  Left to itself the
// compiler merges them into one shared block fed by register moves; these opaque one-instruction
// helpers keep every handler a straight run of arithmetic on its own registers.
__device__ __forceinline__ float op_add(float x, float y) { float r; asm volatile("add.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(x), "f"(y)); return r; }
__device__ __forceinline__ float op_sub(float x, float y) { float r; asm volatile("sub.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(x), "f"(y)); return r; }
__device__ __forceinline__ float op_mul(float x, float y) { float r; asm volatile("mul.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(x), "f"(y)); return r; }
__device__ __forceinline__ float op_fma(float x, float y, float z) { float r; asm volatile("fma.rn.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(x), "f"(y), "f"(z)); return r; }
__device__ __forceinline__ float op_neg(float x) { float r; asm volatile("neg.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float op_mov(float x) { float r; asm volatile("mov.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// One copy of every slow elementary function in the kernel image.
static __device__ __noinline__ float apply_fn(int fn, float x, int n)
{
    switch (fn) {
    case F_EXP: return expf(x);
    case F_LOG: return logf(x);
    case F_SIN: return sinf(x);
    case F_COS: return cosf(x);
    case F_TANH: return tanhf(x);
    case F_SINH: return sinhf(x);
    case F_COSH: return coshf(x);
    default: {   // F_POWI: x ** n by repeated squaring
        unsigned m = n < 0 ? (unsigned)(-n) : (unsigned)n;
        float r = 1.f, b = x;
        while (m) { if (m & 1u) r *= b; b *= b; m >>= 1; }
        return n < 0 ? 1.f / r : r;
    }
    }
}

// Inline versions of the functions that dominate element-wise kernels; everything else goes
// through apply_fn.  Sine and cosine: Cody-Waite reduction by multiples of pi/2 (three-part
// constant, exact first step) and the degree-7 / degree-8 polynomials of the remainder on
// [-pi/4, pi/4]; arguments of 8192 and beyond, infinities and NaN take the library routine (the
// function word tests all values of a thread at once, so that the usual case has no branch per value).
__device__ __forceinline__ float fast_sincos(float x, int quarter)
{
    const float k = rintf(x * 0.636619772367581f);
    float r = fmaf(k, -1.5703125f, x);
    r = fmaf(k, -4.837512969970703125e-4f, r);
    r = fmaf(k, -7.54978995489188216e-8f, r);
    const int q = (int)k + quarter;
    const float r2 = r * r;
    const float sn = fmaf(r * r2, fmaf(r2, fmaf(r2, -1.9515295891e-4f, 8.3321608736e-3f), -1.6666654611e-1f), r);
    const float cs = fmaf(r2 * r2, fmaf(r2, fmaf(r2, 2.443315711809948e-5f, -1.388731625493765e-3f), 4.166664568298827e-2f),
                          fmaf(r2, -0.5f, 1.f));
    const float v = (q & 1) ? cs : sn;
    return (q & 2) ? -v : v;
}
// tanh: odd series below 1/4 (truncation 3e-7 relative), 1 - 2 / (exp(2|x|) + 1) above
__device__ __forceinline__ float fast_tanh(float x)
{
    const float ax = fabsf(x);
    if (ax < 0.25f) {
        const float x2 = x * x;
        return x * fmaf(x2, fmaf(x2, fmaf(x2, -17.f / 315.f, 2.f / 15.f), -1.f / 3.f), 1.f);
    }
    const float e = __expf(2.f * ax);
    return copysignf(1.f - __fdividef(2.f, e + 1.f), x);
}

// Per vector width: NTR temporaries kept in registers (the rest spill to local memory) and the
// usable operand stack depth.  Wide vectors amortise the dispatch cost over more elements and
// pay for it with a shallower stack; the host picks the widest variant a program fits.
#ifndef TAD_RICH_BUILD
#define TAD_RICH_BUILD 0
#endif
template <int TA, int UB>
struct VmCfg {
    static constexpr int E = TA * UB;           // values per thread and operand
    static constexpr int NTR = E >= 16 ? 0 : E >= 8 ? 2 : TADP_NUM_TEMPS;
    // 32 values per thread: the shapes of the product kernels; one operand slot, blocks of 4 warps
    static constexpr int DEPTH = E >= 32 ? 1 : E >= 16 ? TADP_WIDE_DEPTH : STACK;
    // TAD_RICH_BUILD: blocks of 6 warps, two per SM: 168 registers per thread instead of 128
    static constexpr int WARPS = E >= 32 ? 4 : TAD_RICH_BUILD ? 6 : TADP_WARPS_PER_BLOCK;
};

template <int TA, int UB>
struct Vm {
    static constexpr int E = TA * UB;
    float s[VmCfg<TA, UB>::DEPTH][E];
    float tmp[VmCfg<TA, UB>::NTR > 0 ? VmCfg<TA, UB>::NTR : 1][E];
    float acc[E];
    int var[TADP_MAX_VARS];
};

// numerator of a row for vector element 0 of this lane; element t adds t * 32 * coef[lane_var]
__device__ __forceinline__ int row_num(const TadpRow &r, const int (&var)[TADP_MAX_VARS])
{
    unsigned v = (unsigned)r.c0;
#pragma unroll
    for (int k = 0; k < TADP_MAX_VARS; ++k) v += (unsigned)r.coef[k] * (unsigned)var[k];
    return (int)v;
}

__device__ __forceinline__ void set_var(int (&var)[TADP_MAX_VARS], int idx, int value)
{
#pragma unroll
    for (int k = 0; k < TADP_MAX_VARS; ++k) if (k == idx) var[k] = value;
}
__device__ __forceinline__ int get_var(const int (&var)[TADP_MAX_VARS], int idx)
{
    int r = 0;
#pragma unroll
    for (int k = 0; k < TADP_MAX_VARS; ++k) if (k == idx) r = var[k];
    return r;
}

__device__ __forceinline__ unsigned load_offset(const TadpLoad &L, const int (&var)[TADP_MAX_VARS])
{
    unsigned off = (unsigned)L.base;
#pragma unroll
    for (int k = 0; k < TADP_MAX_VARS; ++k) off += (unsigned)L.coef[k] * (unsigned)var[k];
    return off;
}

#define TADV_D0(M, OP) M(OP, 0) M(OP, 1) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6)
#define TADV_D1(M, OP) M(OP, 1) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_D2(M, OP) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_D3(M, OP) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_V8(M, OP) M(OP, 0) M(OP, 1) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_H(OP, K) ((OP) * 8 + (K))
// a handler exists only if the depths it touches fit the variant's stack
#define TADV_CASE(OP, D, TOP) case TADV_H(OP, D): if constexpr ((TOP) <= VmCfg<TA, UB>::DEPTH)

// Runs the program of one work item.  mask0: which vector elements of this lane are live at
// the outermost level.  Returns in live_out the elements that accumulated at least one term.
template <int TA, int UB, bool DEBUG, bool REL>
__device__ __forceinline__ void run_item(const TadpProgram &P, const TadpPointers &ptrs, Vm<TA, UB> &m,
                                         unsigned mask0, int split, unsigned &live_out)
{
    constexpr int T = TA * UB;             // element e = t * UB + u: t along the lane variable, u along the element variable
    const int unroll_var = P.unroll_var;
    unsigned sum_parent = mask0;           // mask outside the sum loop that runs over the element variable
    const int lane_var = P.lane_var;
    unsigned cur = mask0;                 // activity mask of the vector elements at the current loop level
    unsigned mstack[TADP_MAX_ZLOOPS + 1];  // activity mask per loop level
    mstack[0] = mask0;
    unsigned live = 0;
    int loop_hi[TADP_MAX_LOOPS];
    int elo[TADP_MAX_ZLOOPS][T], ehi[TADP_MAX_ZLOOPS][T];
    // per-element start of the relative loop; in shared memory (one column per thread) because it is
    // rarely touched and would otherwise cost T registers in every kernel
    __shared__ int zrel_s[REL ? T : 1][VmCfg<TA, UB>::WARPS * 32];
#define zrel(t) zrel_s[t][threadIdx.x]
    const int rel_var = REL ? P.rel_var : -1;
    constexpr int NTR = VmCfg<TA, UB>::NTR;
    float spill[TADP_MAX_SPILL + TADP_NUM_TEMPS - NTR][T];
#pragma unroll
    for (int t = 0; t < T; ++t) m.acc[t] = 0.f;

    int pc = 0;
    for (;;) {
        const uint2 raw = reinterpret_cast<const uint2 *>(P.code)[pc];   // one 64-bit constant load
        ++pc;
        const int a = (raw.x >> 16) & 0xff;
        const int fn_code = raw.x >> 24;
        const int imm = (int)raw.y;
        switch (raw.x & 0xffffu) {
        case TADV_H(P_END, 0):
            live_out = live;
            return;

#define TADV_CONST(OP, D) TADV_CASE(OP, D, D + 1) { const float c = __int_as_float(imm); _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = op_mov(c); } break;
        TADV_D0(TADV_CONST, P_CONST)
#define TADV_ZERO(OP, D) TADV_CASE(OP, D, D + 1) { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = op_mov(0.f); } break;
        TADV_D0(TADV_ZERO, P_ZERO)

#define TADV_LOAD_BODY(DST_EXPR) { \
            const TadpLoad &L = P.loads[a]; \
            const unsigned off = load_offset(L, m.var); \
            const unsigned lc = (unsigned)L.lane_step; \
            const unsigned uc = UB > 1 ? (unsigned)L.unroll_step : 0u; \
            const float *base = ptrs.in[L.ptr]; \
            if (lc == 0 && uc == 0 && (!REL || L.rel_step == 0) && !DEBUG) { \
                /* the same element for every value of this lane: one load */ \
                const float v = cur ? __ldg(base + off) : 0.f; \
                _Pragma("unroll") for (int t = 0; t < T; ++t) { DST_EXPR; } \
            } else if (UB > 1 && uc == 0 && (!REL || L.rel_step == 0) && !DEBUG) { \
                /* constant along the element variable: one load per lane-variable element */ \
                _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { \
                    const unsigned mm = (cur >> (ta * UB)) & ((1u << UB) - 1u); \
                    const unsigned idx = off + (unsigned)ta * lc;   /* mod 2^32 before it meets the pointer */ \
                    const float v = mm ? __ldg(base + idx) : 0.f; \
                    _Pragma("unroll") for (int u = 0; u < UB; ++u) { const int t = ta * UB + u; DST_EXPR; } \
                } \
            } else if (UB % 4 == 0 && uc == 1 && (!REL || L.rel_step == 0) && !DEBUG && (reinterpret_cast<uintptr_t>(base) & 15u) == 0) { \
                /* contiguous along the element variable: 128-bit loads of this lane's own row */ \
                _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { \
                    const unsigned o = off + (unsigned)ta * lc; \
                    _Pragma("unroll") for (int g4 = 0; g4 < UB / 4; ++g4) { \
                        const unsigned mm = (cur >> (ta * UB + 4 * g4)) & 0xfu; \
                        float q[4]; \
                        if (mm == 0xfu && ((o + 4u * g4) & 3u) == 0) { \
                            const float4 f4 = __ldg(reinterpret_cast<const float4 *>(base + (o + 4u * g4))); \
                            q[0] = f4.x; q[1] = f4.y; q[2] = f4.z; q[3] = f4.w; \
                        } else { \
                            _Pragma("unroll") for (int i = 0; i < 4; ++i) q[i] = ((mm >> i) & 1u) ? __ldg(base + (o + 4u * g4 + i)) : 0.f; \
                        } \
                        _Pragma("unroll") for (int i = 0; i < 4; ++i) { const int t = ta * UB + 4 * g4 + i; const float v = q[i]; DST_EXPR; } \
                    } \
                } \
            } else if (UB > 1 && TA > 1 && lc == 0 && (!REL || L.rel_step == 0) && !DEBUG) { \
                /* the same for every lane and every t: one load per u */ \
                _Pragma("unroll") for (int u = 0; u < UB; ++u) { \
                    unsigned mm = 0; \
                    _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) mm |= (cur >> (ta * UB + u)) & 1u; \
                    const unsigned idx = off + (unsigned)u * uc; \
                    const float v = mm ? __ldg(base + idx) : 0.f; \
                    _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { const int t = ta * UB + u; DST_EXPR; } \
                } \
            } else if (!DEBUG && !REL && cur == (T >= 32 ? 0xffffffffu : ((1u << T) - 1u))) { \
                /* every element live: no per-element predicates */ \
                _Pragma("unroll") for (int t = 0; t < T; ++t) { \
                    const unsigned idx = off + (unsigned)(t / UB) * lc + (unsigned)(t % UB) * uc; \
                    const float v = __ldg(base + idx); \
                    DST_EXPR; \
                } \
            } else { \
                const unsigned rs = REL ? (unsigned)L.rel_step : 0u; \
                _Pragma("unroll") for (int t = 0; t < T; ++t) { \
                    const unsigned idx = off + (unsigned)(t / UB) * lc + (unsigned)(t % UB) * uc + (REL && rs ? rs * (unsigned)zrel(t) : 0u); \
                    bool ok = (cur >> t) & 1u; \
                    if (DEBUG && ok && idx >= (unsigned)L.limit) { ok = false; if (ptrs.debug) atomicCAS(ptrs.debug, 0, 0x10000 + a); } \
                    const float v = ok ? __ldg(base + idx) : 0.f; \
                    DST_EXPR; \
                } \
            } }
#define TADV_LOAD(OP, D) TADV_CASE(OP, D, D + 1) TADV_LOAD_BODY(m.s[D][t] = op_mov(v)) break;
        TADV_D0(TADV_LOAD, P_LOAD)
#define TADV_LDADD(OP, D) TADV_CASE(OP, D, D) TADV_LOAD_BODY(m.s[D - 1][t] = op_add(m.s[D - 1][t], v)) break;
        TADV_D1(TADV_LDADD, P_LDADD)
#define TADV_LDMUL(OP, D) TADV_CASE(OP, D, D) TADV_LOAD_BODY(m.s[D - 1][t] = op_mul(m.s[D - 1][t], v)) break;
        TADV_D1(TADV_LDMUL, P_LDMUL)
#define TADV_LDADDSQ(OP, D) TADV_CASE(OP, D, D) TADV_LOAD_BODY({ const float w2 = op_add(m.s[D - 1][t], v); m.s[D - 1][t] = op_mul(w2, w2); }) break;
        TADV_D1(TADV_LDADDSQ, P_LDADDSQ)

#define TADV_UNARY(D, EXPR) { _Pragma("unroll") for (int t = 0; t < T; ++t) { const float x = m.s[D - 1][t]; m.s[D - 1][t] = (EXPR); } } break;
#define TADV_NEG(OP, D) TADV_CASE(OP, D, D) TADV_UNARY(D, op_neg(x))
        TADV_D1(TADV_NEG, P_NEG)
#define TADV_SQR(OP, D) TADV_CASE(OP, D, D) TADV_UNARY(D, op_mul(x, x))
        TADV_D1(TADV_SQR, P_SQR)
#define TADV_CUBE(OP, D) TADV_CASE(OP, D, D) TADV_UNARY(D, op_mul(op_mul(x, x), x))
        TADV_D1(TADV_CUBE, P_CUBE)
#define TADV_MULC(OP, D) TADV_CASE(OP, D, D) { const float c = __int_as_float(imm); TADV_UNARY(D, op_mul(x, c)) }
        TADV_D1(TADV_MULC, P_MULC)
#define TADV_ADDC(OP, D) TADV_CASE(OP, D, D) { const float c = __int_as_float(imm); TADV_UNARY(D, op_add(x, c)) }
        TADV_D1(TADV_ADDC, P_ADDC)
#define TADV_FN(OP, D) TADV_CASE(OP, D, D) { \
            if (UB > 1 && a) { \
                /* the operand is the same for every u: one evaluation per t, taken from the first live u \
                   (a value sum leaves the elements that are masked off unfinished) */ \
                _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { \
                    float src = m.s[D - 1][ta * UB + UB - 1]; \
                    _Pragma("unroll") for (int u = UB - 2; u >= 0; --u) if ((cur >> (ta * UB + u)) & 1u) src = m.s[D - 1][ta * UB + u]; \
                    const float r = apply_fn(fn_code, src, imm); \
                    _Pragma("unroll") for (int u = 0; u < UB; ++u) m.s[D - 1][ta * UB + u] = r; \
                } \
                break; \
            } \
            switch (fn_code) { \
            case F_EXP: { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 1][t] = __expf(m.s[D - 1][t]); } break; \
            case F_SIN: case F_COS: { \
                const int quarter = fn_code == F_COS ? 1 : 0; \
                float biggest = 0.f; \
                _Pragma("unroll") for (int t = 0; t < T; ++t) biggest = fmaxf(biggest, fabsf(m.s[D - 1][t]) < 8192.f ? 0.f : 1.f); \
                if (biggest == 0.f) { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 1][t] = fast_sincos(m.s[D - 1][t], quarter); } \
                else { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 1][t] = apply_fn(fn_code, m.s[D - 1][t], imm); } \
            } break; \
            case F_TANH: { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 1][t] = fast_tanh(m.s[D - 1][t]); } break; \
            default: { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 1][t] = apply_fn(fn_code, m.s[D - 1][t], imm); } break; \
            } } break;
        TADV_D1(TADV_FN, P_FN)

#define TADV_BINARY(D, EXPR) { _Pragma("unroll") for (int t = 0; t < T; ++t) { const float x = m.s[D - 2][t], y = m.s[D - 1][t]; m.s[D - 2][t] = (EXPR); } } break;
#define TADV_ADD(OP, D) TADV_CASE(OP, D, D) TADV_BINARY(D, op_add(x, y))
        TADV_D2(TADV_ADD, P_ADD)
        // summand into the accumulator of a value sum; elements masked off (the tail of a sum that
        // runs over the element variable) leave it unchanged
#define TADV_SUMADD(OP, D) TADV_CASE(OP, D, D) { _Pragma("unroll") for (int t = 0; t < T; ++t) if (UB == 1 || ((cur >> t) & 1u)) m.s[D - 2][t] = op_add(m.s[D - 2][t], m.s[D - 1][t]); } break;
        TADV_D2(TADV_SUMADD, P_SUMADD)
        // summand into the accumulator and the end of the (ordinary) sum loop in one word
#define TADV_SUMEND(OP, D) TADV_CASE(OP, D, D) { \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 2][t] = op_add(m.s[D - 2][t], m.s[D - 1][t]); \
            const TadpLoop &L = P.loops[a]; \
            const int k = get_var(m.var, L.var) + 1; \
            if (k <= L.const_hi) { set_var(m.var, L.var, k); pc = imm; } } break;
        TADV_D2(TADV_SUMEND, P_SUMEND)
        // closes a sum over the element variable: add up the UB partial sums, replicate the result
#define TADV_HSUM(OP, D) TADV_CASE(OP, D, D) { \
            _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { \
                float sum = m.s[D - 1][ta * UB]; \
                _Pragma("unroll") for (int u = 1; u < UB; ++u) sum = op_add(sum, m.s[D - 1][ta * UB + u]); \
                _Pragma("unroll") for (int u = 0; u < UB; ++u) m.s[D - 1][ta * UB + u] = op_mov(sum); \
            } } break;
        TADV_D1(TADV_HSUM, P_HSUM)
#define TADV_SUB(OP, D) TADV_CASE(OP, D, D) TADV_BINARY(D, op_sub(x, y))
        TADV_D2(TADV_SUB, P_SUB)
#define TADV_MUL(OP, D) TADV_CASE(OP, D, D) TADV_BINARY(D, op_mul(x, y))
        TADV_D2(TADV_MUL, P_MUL)
#define TADV_DIV(OP, D) TADV_CASE(OP, D, D) TADV_BINARY(D, x / y)
        TADV_D2(TADV_DIV, P_DIV)
#define TADV_FMA(OP, D) TADV_CASE(OP, D, D) { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 3][t] = op_fma(m.s[D - 3][t], m.s[D - 2][t], m.s[D - 1][t]); } break;
        TADV_D3(TADV_FMA, P_FMA)

#define TADV_TEMP_CASE(KK, STMT_REG, STMT_SPILL) case KK: if constexpr (KK < NTR) { constexpr int K = KK; STMT_REG } else { const int K = KK - NTR; STMT_SPILL } break;
#define TADV_TEMP_SWITCH(STMT_REG, STMT_SPILL) TADV_TEMP_SWITCH_ON(a, STMT_REG, STMT_SPILL)
#define TADV_TEMP_SWITCH_ON(SEL, STMT_REG, STMT_SPILL) \
            switch (SEL) { \
            TADV_TEMP_CASE(0, STMT_REG, STMT_SPILL) TADV_TEMP_CASE(1, STMT_REG, STMT_SPILL) \
            TADV_TEMP_CASE(2, STMT_REG, STMT_SPILL) TADV_TEMP_CASE(3, STMT_REG, STMT_SPILL) \
            TADV_TEMP_CASE(4, STMT_REG, STMT_SPILL) TADV_TEMP_CASE(5, STMT_REG, STMT_SPILL) \
            TADV_TEMP_CASE(6, STMT_REG, STMT_SPILL) TADV_TEMP_CASE(7, STMT_REG, STMT_SPILL) \
            default: { const int K = (SEL) - NTR; STMT_SPILL } break; }
#define TADV_LDT(OP, D) TADV_CASE(OP, D, D + 1) { TADV_TEMP_SWITCH( \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = op_mov(m.tmp[K][t]);, \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = spill[K][t];) } break;
        TADV_D0(TADV_LDT, P_LDT)
#define TADV_STT(OP, D) TADV_CASE(OP, D, D) { TADV_TEMP_SWITCH( \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.tmp[K][t] = op_mov(m.s[D - 1][t]);, \
            _Pragma("unroll") for (int t = 0; t < T; ++t) spill[K][t] = m.s[D - 1][t];) } break;
        TADV_D1(TADV_STT, P_STT)

#define TADV_FMAT(OP, D) TADV_CASE(OP, D, D) { TADV_TEMP_SWITCH( \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 2][t] = op_fma(m.s[D - 2][t], m.tmp[K][t], m.s[D - 1][t]);, \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 2][t] = op_fma(m.s[D - 2][t], spill[K][t], m.s[D - 1][t]);) } break;
        TADV_D2(TADV_FMAT, P_FMAT)
#define TADV_ACC(OP, D) TADV_CASE(OP, D, D) { _Pragma("unroll") for (int t = 0; t < T; ++t) if ((cur >> t) & 1u) m.acc[t] = op_add(m.acc[t], m.s[D - 1][t]); live |= cur; } break;
        TADV_D1(TADV_ACC, P_ACC)
#define TADV_SCALE(OP, D) TADV_CASE(OP, D, D) { _Pragma("unroll") for (int t = 0; t < T; ++t) m.acc[t] = op_mul(m.acc[t], m.s[D - 1][t]); } break;
        TADV_D1(TADV_SCALE, P_SCALE)
#define TADV_MACC(OP, D) TADV_CASE(OP, D, D) { _Pragma("unroll") for (int t = 0; t < T; ++t) if ((cur >> t) & 1u) m.acc[t] = op_fma(m.s[D - 2][t], m.s[D - 1][t], m.acc[t]); live |= cur; } break;
        TADV_D2(TADV_MACC, P_MACC)

        // ---- loop control: the handler number carries the loop variable ----
#define TADV_SLOOP(OP, V) case TADV_H(OP, V): { const TadpLoop &L = P.loops[a]; if (L.const_lo > L.const_hi) pc = imm; else m.var[V] = L.const_lo; } break;
        TADV_V8(TADV_SLOOP, P_SLOOP)
#define TADV_SEND(OP, V) case TADV_H(OP, V): { const int k = m.var[V] + 1; if (k <= P.loops[a].const_hi) { m.var[V] = k; pc = imm; } } break;
        TADV_V8(TADV_SEND, P_SEND)
        // the sum whose index is the element variable: UB summands per trip, tail masked
#define TADV_USLOOP(OP, V) case TADV_H(OP, V): { \
            const TadpLoop &L = P.loops[a]; \
            if (L.const_lo > L.const_hi) pc = imm; \
            else { \
                m.var[V] = L.const_lo; sum_parent = cur; \
                unsigned mk = 0; \
                _Pragma("unroll") for (int t = 0; t < T; ++t) if (L.const_lo + (t % UB) <= L.const_hi) mk |= 1u << t; \
                cur = sum_parent & mk; \
            } } break;
        TADV_V8(TADV_USLOOP, P_USLOOP)
#define TADV_USEND(OP, V) case TADV_H(OP, V): { \
            const int k = m.var[V] + UB; const int hi = P.loops[a].const_hi; \
            if (k <= hi) { \
                m.var[V] = k; \
                unsigned mk = 0; \
                _Pragma("unroll") for (int t = 0; t < T; ++t) if (k + (t % UB) <= hi) mk |= 1u << t; \
                cur = sum_parent & mk; pc = imm; \
            } else cur = sum_parent; } break;
        TADV_V8(TADV_USEND, P_USEND)

#define TADV_ZLOOP_BODY { \
            const TadpLoop &L = P.loops[a]; const int V = L.var; \
            const int lvl = L.mask_level; \
            const unsigned parent = mstack[lvl - 1]; \
            int wlo, whi; \
            if (L.is_lane || !L.depends_on_lane) { \
                int lo = INT_MIN, hi = INT_MAX; \
                for (int r = 0; r < L.n_lower; ++r) { const TadpRow &R = P.rows[L.lower0 + r]; const int nmr = row_num(R, m.var); lo = max(lo, R.den == 1 ? nmr : ceil_div_i(nmr, R.den)); } \
                for (int r = 0; r < L.n_upper; ++r) { const TadpRow &R = P.rows[L.upper0 + r]; const int nmr = row_num(R, m.var); hi = min(hi, R.den == 1 ? nmr : floor_div_i(nmr, R.den)); } \
                wlo = lo; whi = hi; \
                if (L.is_split && lo <= hi) { \
                    /* this warp's contiguous share of the range (fixed chunking: repeatable sums) */ \
                    const int chunk = (hi - lo + L.split_n) / L.split_n; \
                    wlo = lo + ((split / L.split_div) % L.split_n) * chunk; whi = min(hi, wlo + chunk - 1); \
                } \
                if (__ballot_sync(0xffffffffu, parent != 0) == 0) { wlo = 1; whi = 0; } \
            } else { \
                int lo_w = INT_MAX, hi_w = INT_MIN; \
                _Pragma("unroll") for (int t = 0; t < T; ++t) { elo[lvl - 1][t] = INT_MIN; ehi[lvl - 1][t] = INT_MAX; } \
                for (int r = 0; r < L.n_lower; ++r) { \
                    const TadpRow &R = P.rows[L.lower0 + r]; \
                    const int nmr = row_num(R, m.var); const int step = R.coef[lane_var] * 32; \
                    const int ustep = (UB > 1 && unroll_var >= 0) ? R.coef[unroll_var] : 0; \
                    const int rstep = rel_var >= 0 ? R.coef[rel_var] : 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) { int v = nmr + (t / UB) * step + (t % UB) * ustep + (REL && rstep ? rstep * zrel(t) : 0); v = R.den == 1 ? v : ceil_div_i(v, R.den); elo[lvl - 1][t] = max(elo[lvl - 1][t], v); } \
                } \
                for (int r = 0; r < L.n_upper; ++r) { \
                    const TadpRow &R = P.rows[L.upper0 + r]; \
                    const int nmr = row_num(R, m.var); const int step = R.coef[lane_var] * 32; \
                    const int ustep = (UB > 1 && unroll_var >= 0) ? R.coef[unroll_var] : 0; \
                    const int rstep = rel_var >= 0 ? R.coef[rel_var] : 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) { int v = nmr + (t / UB) * step + (t % UB) * ustep + (REL && rstep ? rstep * zrel(t) : 0); v = R.den == 1 ? v : floor_div_i(v, R.den); ehi[lvl - 1][t] = min(ehi[lvl - 1][t], v); } \
                } \
                _Pragma("unroll") for (int t = 0; t < T; ++t) \
                    if (((parent >> t) & 1u) && elo[lvl - 1][t] <= ehi[lvl - 1][t]) { lo_w = min(lo_w, elo[lvl - 1][t]); hi_w = max(hi_w, ehi[lvl - 1][t]); } \
                if (L.is_split) { \
                    /* the union of the warp's element ranges is divided into zsplit contiguous shares, the same for \
                       every element, so that the elements of a share walk it together (fixed chunking: repeatable sums) */ \
                    _Pragma("unroll") for (int o = 16; o > 0; o >>= 1) { lo_w = min(lo_w, __shfl_xor_sync(0xffffffffu, lo_w, o)); hi_w = max(hi_w, __shfl_xor_sync(0xffffffffu, hi_w, o)); } \
                    if (lo_w <= hi_w) { \
                        const int chunk = (hi_w - lo_w + L.split_n) / L.split_n; \
                        const int slo = lo_w + ((split / L.split_div) % L.split_n) * chunk, shi = min(hi_w, slo + chunk - 1); \
                        lo_w = INT_MAX; hi_w = INT_MIN; \
                        _Pragma("unroll") for (int t = 0; t < T; ++t) { \
                            elo[lvl - 1][t] = max(elo[lvl - 1][t], slo); ehi[lvl - 1][t] = min(ehi[lvl - 1][t], shi); \
                            if (((parent >> t) & 1u) && elo[lvl - 1][t] <= ehi[lvl - 1][t]) { lo_w = min(lo_w, elo[lvl - 1][t]); hi_w = max(hi_w, ehi[lvl - 1][t]); } \
                        } \
                    } \
                } \
                if (REL && L.is_relative) { \
                    /* trip r visits lo_e + r: the warp runs as many trips as its longest element range */ \
                    int len = 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) { \
                        if (((parent >> t) & 1u) && elo[lvl - 1][t] <= ehi[lvl - 1][t]) len = max(len, ehi[lvl - 1][t] - elo[lvl - 1][t] + 1); \
                        else { ehi[lvl - 1][t] = -1; elo[lvl - 1][t] = 0; } \
                        zrel(t) = elo[lvl - 1][t]; ehi[lvl - 1][t] -= elo[lvl - 1][t]; elo[lvl - 1][t] = 0; \
                    } \
                    _Pragma("unroll") for (int o = 16; o > 0; o >>= 1) len = max(len, __shfl_xor_sync(0xffffffffu, len, o)); \
                    lo_w = 0; hi_w = len - 1; \
                } else { \
                _Pragma("unroll") for (int o = 16; o > 0; o >>= 1) { lo_w = min(lo_w, __shfl_xor_sync(0xffffffffu, lo_w, o)); hi_w = max(hi_w, __shfl_xor_sync(0xffffffffu, hi_w, o)); } \
                } \
                wlo = lo_w; whi = hi_w; \
            } \
            if (wlo > whi) { pc = imm; if (REL && L.is_relative) { _Pragma("unroll") for (int t = 0; t < T; ++t) zrel(t) = 0; } } \
            else { \
                loop_hi[a] = whi; \
                unsigned mk; \
                if (L.is_lane) { \
                    const int z = wlo + (int)(threadIdx.x & 31u); \
                    set_var(m.var, V, z); \
                    mk = 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (z + 32 * (t / UB) <= whi) mk |= 1u << t; \
                    mk &= parent; \
                } else { \
                    set_var(m.var, V, wlo); \
                    mk = parent; \
                    if (L.depends_on_lane) { \
                        mk = 0; \
                        _Pragma("unroll") for (int t = 0; t < T; ++t) if (elo[lvl - 1][t] <= wlo && wlo <= ehi[lvl - 1][t]) mk |= 1u << t; \
                        mk &= parent; \
                    } \
                } \
                cur = mk; \
                mstack[lvl] = mk; \
            } }

#define TADV_ZEND_BODY { \
            const TadpLoop &L = P.loops[a]; const int V = L.var; \
            const int lvl = L.mask_level; \
            const unsigned parent = mstack[lvl - 1]; \
            const int whi = loop_hi[a]; \
            const int z = get_var(m.var, V) + (L.is_lane ? 32 * TA : 1); \
            const int zbase = L.is_lane ? z - (int)(threadIdx.x & 31u) : z; \
            if (zbase <= whi) { \
                set_var(m.var, V, z); \
                unsigned mk; \
                if (L.is_lane) { \
                    mk = 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (z + 32 * (t / UB) <= whi) mk |= 1u << t; \
                    mk &= parent; \
                } else if (L.depends_on_lane) { \
                    mk = 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (elo[lvl - 1][t] <= z && z <= ehi[lvl - 1][t]) mk |= 1u << t; \
                    mk &= parent; \
                } else mk = parent; \
                cur = mk; \
                mstack[lvl] = mk; \
                pc = imm; \
            } else { \
                cur = parent; \
                if (REL && L.is_relative) { _Pragma("unroll") for (int t = 0; t < T; ++t) zrel(t) = 0; set_var(m.var, V, 0); } \
            } }
        // ---- fused innermost loop: all trips of the loop run here, without a dispatch per word ----
        // X = s[SUMMODE], Y = s[SUMMODE + 1], invariants in the two topmost stack registers; a value sum
        // accumulates into s[0], a gradient loop into acc.  Load offsets advance by a fixed step per trip.
#define TADV_XSTEP(CODE, EXPR) case CODE: { _Pragma("unroll") for (int t = 0; t < T; ++t) { const float x = m.s[XI][t]; const float y = m.s[YI][t]; (void)y; m.s[XI][t] = (EXPR); } } break;
#define TADV_XC_SET(t, x) m.s[XI][t] = op_mov(x);
#define TADV_XC_ADD(t, x) m.s[XI][t] = op_add(m.s[XI][t], (x));
#define TADV_XC_MUL(t, x) m.s[XI][t] = op_mul(m.s[XI][t], (x));
#define TADV_XC_ADDSQ(t, x) { const float w2 = op_add(m.s[XI][t], (x)); m.s[XI][t] = op_mul(w2, w2); }
        // fetches one load of the body in the manner the host chose and hands every element's value to COMBINE;
        // ALL: every element of the thread is live (no predicates, signed 64-bit addressing from element 0)
#define TADV_XF_REL(COMBINE, ALL) { \
                                /* inside a relative loop: every element reads at its own position of that loop */ \
                                _Pragma("unroll") for (int t = 0; t < T; ++t) { \
                                    const unsigned idx = off + (unsigned)(t / UB) * lc + (unsigned)(t % UB) * uc + rs * (unsigned)zrel(t); \
                                    const float x = (ALL || ((cur >> t) & 1u)) ? __ldg(base + idx) : 0.f; COMBINE(t, x) } }
#define TADV_XF_ONE(COMBINE, ALL) { \
                                const float x = (ALL || cur) ? __ldg(base + off) : 0.f; \
                                _Pragma("unroll") for (int t = 0; t < T; ++t) { COMBINE(t, x) } }
#define TADV_XF_PER_T(COMBINE, ALL) { if constexpr (UB > 1) { \
                                _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { \
                                    const unsigned mm = ALL ? 1u : (cur >> (ta * UB)) & ((1u << UB) - 1u); \
                                    const unsigned idx = off + (unsigned)ta * lc; \
                                    const float x = mm ? __ldg(base + idx) : 0.f; \
                                    _Pragma("unroll") for (int u = 0; u < UB; ++u) { COMBINE(ta * UB + u, x) } \
                                } } }
#define TADV_XF_PER_U(COMBINE, ALL) { if constexpr (UB > 1) { \
                                _Pragma("unroll") for (int u = 0; u < UB; ++u) { \
                                    unsigned mm = ALL ? 1u : 0u; \
                                    if (!ALL) { _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) mm |= (cur >> (ta * UB + u)) & 1u; } \
                                    const unsigned idx = off + (unsigned)u * uc; \
                                    const float x = mm ? __ldg(base + idx) : 0.f; \
                                    _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { COMBINE(ta * UB + u, x) } \
                                } } }
#define TADV_XF_EACH(COMBINE, ALL) { \
                                if (ALL) { \
                                    const float *p0 = base + off; \
                                    _Pragma("unroll") for (int t = 0; t < T; ++t) { const float x = __ldg(p0 + ((t / UB) * (int)lc + (t % UB) * (int)uc)); COMBINE(t, x) } \
                                } else { \
                                    _Pragma("unroll") for (int t = 0; t < T; ++t) { const unsigned idx = off + (unsigned)(t / UB) * lc + (unsigned)(t % UB) * uc; const float x = ((cur >> t) & 1u) ? __ldg(base + idx) : 0.f; COMBINE(t, x) } \
                                } }
        // rows of four along the element variable as 128-bit loads when the pointer allows, else element by element
#define TADV_XF_ROW(COMBINE, ALL) { \
                                bool rows_done = false; \
                                if constexpr (UB > 1 && UB % 4 == 0) { \
                                if ((reinterpret_cast<uintptr_t>(base) & 15u) == 0) { \
                                    rows_done = true; \
                                    _Pragma("unroll") for (int ta = 0; ta < TA; ++ta) { \
                                        const unsigned ob = off + (unsigned)ta * lc; \
                                        _Pragma("unroll") for (int g4 = 0; g4 < UB / 4; ++g4) { \
                                            const unsigned mm = ALL ? 0xfu : (cur >> (ta * UB + 4 * g4)) & 0xfu; \
                                            float q[4]; \
                                            if (mm == 0xfu && ((ob + 4u * g4) & 3u) == 0) { \
                                                const float4 f4 = __ldg(reinterpret_cast<const float4 *>(base + (ob + 4u * g4))); \
                                                q[0] = f4.x; q[1] = f4.y; q[2] = f4.z; q[3] = f4.w; \
                                            } else { \
                                                _Pragma("unroll") for (int i = 0; i < 4; ++i) q[i] = ((mm >> i) & 1u) ? __ldg(base + (ob + 4u * g4 + i)) : 0.f; \
                                            } \
                                            _Pragma("unroll") for (int i = 0; i < 4; ++i) { COMBINE(ta * UB + 4 * g4 + i, q[i]) } \
                                        } \
                                    } \
                                } } \
                                if (!rows_done) TADV_XF_EACH(COMBINE, ALL) }
#define TADV_XFETCH(COMBINE, ALL) \
                            if (REL && rs != 0) TADV_XF_REL(COMBINE, ALL) \
                            else switch (fk) { \
                            case BF_ONE: TADV_XF_ONE(COMBINE, ALL) break; \
                            case BF_PER_T: TADV_XF_PER_T(COMBINE, ALL) break; \
                            case BF_PER_U: TADV_XF_PER_U(COMBINE, ALL) break; \
                            case BF_ROW: TADV_XF_ROW(COMBINE, ALL) break; \
                            default: TADV_XF_EACH(COMBINE, ALL) break; \
                            }
        // one dispatch per load step: fetch kind and combine together select the code
#define TADV_XF_CASES(KIND, FETCH, ALL) \
                            case (KIND) * 4 + 0: FETCH(TADV_XC_SET, ALL) break; \
                            case (KIND) * 4 + 1: FETCH(TADV_XC_ADD, ALL) break; \
                            case (KIND) * 4 + 2: FETCH(TADV_XC_MUL, ALL) break; \
                            case (KIND) * 4 + 3: FETCH(TADV_XC_ADDSQ, ALL) break;
        // the steps of one trip and the term that closes it
#define TADV_XTRIP(SUMMODE, ALL) { \
                unsigned w0 = steps.x, w1 = steps.y; \
                for (;;) { \
                    const unsigned c = w0 & 0xffu; \
                    if (c == 0) break; \
                    w0 = __funnelshift_r(w0, w1, 8); w1 >>= 8; \
                    if (c & 0x80u) { \
                        const unsigned j = c & 3u; \
                        const unsigned off = TADV_XSEL(j, xo); \
                        const unsigned lc = TADV_XSEL(j, xlc); \
                        const unsigned uc = TADV_XSEL(j, xuc); \
                        const unsigned rs = REL ? TADV_XSEL(j, xrs) : 0u; (void)rs; \
                        const float *base = TADV_XSEL(j, xbase); \
                        if (REL && rs != 0) { \
                            switch ((c >> 2) & 3u) { TADV_XF_CASES(0, TADV_XF_REL, ALL) } \
                        } else switch ((c >> 2) & 0x1fu) {   /* fetch kind x 4 + combine */ \
                        TADV_XF_CASES(BF_ONE, TADV_XF_ONE, ALL) \
                        TADV_XF_CASES(BF_PER_T, TADV_XF_PER_T, ALL) \
                        TADV_XF_CASES(BF_PER_U, TADV_XF_PER_U, ALL) \
                        TADV_XF_CASES(BF_ROW, TADV_XF_ROW, ALL) \
                        TADV_XF_CASES(BF_EACH, TADV_XF_EACH, ALL) \
                        default: break; \
                        } \
                    } else { \
                        switch (c) { \
                        case BS_PUSH: { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[YI][t] = op_mov(m.s[XI][t]); } break; \
                        TADV_XSTEP(BS_NEG, op_neg(x)) TADV_XSTEP(BS_SQR, op_mul(x, x)) TADV_XSTEP(BS_CUBE, op_mul(op_mul(x, x), x)) \
                        TADV_XSTEP(BS_ADDY, op_add(y, x)) TADV_XSTEP(BS_SUBY, op_sub(y, x)) TADV_XSTEP(BS_MULY, op_mul(y, x)) TADV_XSTEP(BS_DIVY, y / x) \
                        TADV_XSTEP(BS_LDI0, op_mov(m.s[I0][t])) TADV_XSTEP(BS_LDI1, op_mov(m.s[I1][t])) \
                        TADV_XSTEP(BS_MULI0, op_mul(x, m.s[I0][t])) TADV_XSTEP(BS_MULI1, op_mul(x, m.s[I1][t])) \
                        TADV_XSTEP(BS_ADDI0, op_add(x, m.s[I0][t])) TADV_XSTEP(BS_ADDI1, op_add(x, m.s[I1][t])) \
                        TADV_XSTEP(BS_FMAYI0, op_fma(y, m.s[I0][t], x)) \
                        default: { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[XI][t] = op_fma(m.s[YI][t], m.s[I1][t], m.s[XI][t]); } break; \
                        } \
                    } \
                } \
                if (SUMMODE) { \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (ALL || UB == 1 || ((cur >> t) & 1u)) \
                        m.s[0][t] = term ? op_fma(m.s[YI][t], m.s[XI][t], m.s[0][t]) : op_add(m.s[0][t], m.s[XI][t]); \
                } else { \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (ALL || ((cur >> t) & 1u)) \
                        m.acc[t] = term ? op_fma(m.s[YI][t], m.s[XI][t], m.acc[t]) : op_add(m.acc[t], m.s[XI][t]); \
                    live |= cur; \
                } }
#define TADV_XSEL(j, A) ((j) == 0 ? A[0] : (j) == 1 ? A[1] : (j) == 2 ? A[2] : A[3])
        // ---- product loops of the 32-value shapes: S += P * Q, P (one value per u, or one per t) into a small
        // buffer, Q multiplied in and accumulated value by value as it arrives; nothing but S has 32 entries ----
#define TADV_DC_PU(t, x) pu[(t) % UB] = (x);
#define TADV_DC_PT(t, x) pt[(t) / UB] = (x);
#define TADV_DC_ACC(t, p, x, ALL) if (ALL || (SM && UB == 1) || ((cur >> (t)) & 1u)) SS[t] = op_fma((p), (x), SS[t]);
#define TADV_DC_QU_T(t, x) TADV_DC_ACC(t, pu[(t) % UB], x, true)
#define TADV_DC_QT_T(t, x) TADV_DC_ACC(t, pt[(t) / UB], x, true)
#define TADV_DC_QU_F(t, x) TADV_DC_ACC(t, pu[(t) % UB], x, false)
#define TADV_DC_QT_F(t, x) TADV_DC_ACC(t, pt[(t) / UB], x, false)
#define TADV_DOT_SLOT(J) \
                const unsigned fk = (unsigned)B.dot_fk[J]; const unsigned off = xo[J], lc = xlc[J], uc = xuc[J]; \
                const unsigned rs = 0u; (void)rs; const float *base = xbase[J];
#define TADV_DOTTRIP(ALL, SUF) { \
                float pu[UB], pt[TA]; \
                if (pcls == 0) { \
                    { TADV_DOT_SLOT(0) TADV_XFETCH(TADV_DC_PU, ALL) } \
                    { TADV_DOT_SLOT(1) TADV_XFETCH(TADV_DC_QU_##SUF, ALL) } \
                } else { \
                    { TADV_DOT_SLOT(0) TADV_XFETCH(TADV_DC_PT, ALL) } \
                    { TADV_DOT_SLOT(1) TADV_XFETCH(TADV_DC_QT_##SUF, ALL) } \
                } \
                if (!SM) live |= cur; }
#define TADV_XLOOP_WIDE(SUMMODE) if constexpr (!DEBUG && !REL && T >= 32) { \
            constexpr bool SM = (SUMMODE) != 0; \
            float (&SS)[T] = SM ? m.s[0] : m.acc; \
            const TadpBody &B = P.bodies[imm]; \
            const TadpLoop &L = P.loops[a]; \
            const int V = L.var; \
            const int kind = B.loop_kind; \
            const int pcls = B.dot_pclass; \
            int z = get_var(m.var, V); \
            const int lane = (int)(threadIdx.x & 31u); \
            const int dz = kind == BL_USUM ? UB : kind == BL_Z_LANE ? 32 * TA : 1; \
            const int hi = kind <= BL_USUM ? L.const_hi : loop_hi[a]; \
            const int lvl = L.mask_level; \
            const unsigned parent = kind == BL_SUM ? cur : kind == BL_USUM ? sum_parent : mstack[lvl - 1]; \
            unsigned xo[2], xst[2], xlc[2], xuc[2]; \
            const float *xbase[2]; \
            _Pragma("unroll") for (int j = 0; j < 2; ++j) { \
                const TadpLoad &Ld = P.loads[B.load[j]]; \
                xo[j] = load_offset(Ld, m.var); xst[j] = (unsigned)Ld.coef[V] * (unsigned)dz; \
                xlc[j] = (unsigned)Ld.lane_step; xuc[j] = UB > 1 ? (unsigned)Ld.unroll_step : 0u; \
                xbase[j] = ptrs.in[Ld.ptr]; \
            } \
            constexpr unsigned FULL = 0xffffffffu; \
            if (UB > 1 && pcls == 0 && B.dot_fk[0] == BF_PER_U && B.dot_fk[1] == BF_PER_T && cur == FULL && (kind == BL_SUM || kind == BL_Z)) { \
                /* outer product, every element live in every trip: one value per u (the same for all lanes) times one \
                   value per t.  The operands of the next trip are loaded while the multiply-adds of this one run. */ \
                float pu[UB], pt[TA], nt[TA]; \
                _Pragma("unroll") for (int u = 0; u < UB; ++u) pu[u] = __ldg(xbase[0] + (xo[0] + (unsigned)u * xuc[0])); \
                _Pragma("unroll") for (int t = 0; t < TA; ++t) pt[t] = __ldg(xbase[1] + (xo[1] + (unsigned)t * xlc[1])); \
                for (;;) { \
                    ++z; \
                    const bool more = z <= hi; \
                    if (more) { \
                        xo[0] += xst[0]; xo[1] += xst[1]; \
                        _Pragma("unroll") for (int t = 0; t < TA; ++t) nt[t] = __ldg(xbase[1] + (xo[1] + (unsigned)t * xlc[1])); \
                    } \
                    _Pragma("unroll") for (int u = 0; u < UB; ++u) { \
                        _Pragma("unroll") for (int t = 0; t < TA; ++t) SS[t * UB + u] = fmaf(pu[u], pt[t], SS[t * UB + u]); \
                        /* this per-u value is used up: its register takes the value of the next trip */ \
                        if (more) pu[u] = __ldg(xbase[0] + (xo[0] + (unsigned)u * xuc[0])); \
                    } \
                    if (!more) break; \
                    _Pragma("unroll") for (int t = 0; t < TA; ++t) pt[t] = nt[t]; \
                } \
                if (!SM) live |= cur; \
            } else if (UB > 1 && pcls == 1 && B.dot_fk[0] == BF_PER_T && (B.dot_fk[1] == BF_EACH || B.dot_fk[1] == BF_ROW) && cur == FULL && \
                       (kind == BL_SUM || kind == BL_Z)) { \
                /* one value per t times one value per element, every element live in every trip */ \
                float pt[TA], nt[TA]; \
                _Pragma("unroll") for (int t = 0; t < TA; ++t) pt[t] = __ldg(xbase[0] + (xo[0] + (unsigned)t * xlc[0])); \
                for (;;) { \
                    const unsigned qo = xo[1]; \
                    ++z; \
                    const bool more = z <= hi; \
                    if (more) { \
                        xo[0] += xst[0]; xo[1] += xst[1]; \
                        _Pragma("unroll") for (int t = 0; t < TA; ++t) nt[t] = __ldg(xbase[0] + (xo[0] + (unsigned)t * xlc[0])); \
                    } \
                    _Pragma("unroll") for (int t = 0; t < TA; ++t) { \
                        float q[UB]; \
                        _Pragma("unroll") for (int u = 0; u < UB; ++u) q[u] = __ldg(xbase[1] + (qo + (unsigned)t * xlc[1] + (unsigned)u * xuc[1])); \
                        _Pragma("unroll") for (int u = 0; u < UB; ++u) SS[t * UB + u] = fmaf(pt[t], q[u], SS[t * UB + u]); \
                    } \
                    if (!more) break; \
                    _Pragma("unroll") for (int t = 0; t < TA; ++t) pt[t] = nt[t]; \
                } \
                if (!SM) live |= cur; \
            } else \
            for (;;) { \
                if (cur == FULL) TADV_DOTTRIP(true, T) else TADV_DOTTRIP(false, F) \
                z += dz; \
                const int zb = kind == BL_Z_LANE ? z - lane : z; \
                if (zb > hi) break; \
                xo[0] += xst[0]; xo[1] += xst[1]; \
                if (kind == BL_Z_MASKED) { \
                    unsigned mk = 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (elo[lvl - 1][t] <= z && z <= ehi[lvl - 1][t]) mk |= 1u << t; \
                    cur = parent & mk; \
                } else if (zb + dz - 1 > hi) { \
                    unsigned mk = 0; \
                    if (kind == BL_USUM) { _Pragma("unroll") for (int t = 0; t < T; ++t) if (z + (t % UB) <= hi) mk |= 1u << t; } \
                    else { _Pragma("unroll") for (int t = 0; t < T; ++t) if (z + 32 * (t / UB) <= hi) mk |= 1u << t; } \
                    cur = parent & mk; \
                } \
            } \
            cur = parent; \
        } else
#define TADV_XLOOP(SUMMODE) case TADV_H(P_XLOOP, SUMMODE): TADV_XLOOP_WIDE(SUMMODE) if constexpr (!DEBUG && (SUMMODE) + 2 <= VmCfg<TA, UB>::DEPTH) { \
            constexpr int DEPTH = VmCfg<TA, UB>::DEPTH; \
            constexpr int XI = (SUMMODE), YI = XI + 1, I0 = DEPTH - 1, I1 = DEPTH >= 2 ? DEPTH - 2 : 0; \
            const TadpBody &B = P.bodies[imm]; \
            const TadpLoop &L = P.loops[a]; \
            const int V = L.var; \
            const int kind = B.loop_kind; \
            _Pragma("unroll") for (int q = 0; q < 2; ++q) { \
                const int ik = B.inv_kind[q]; \
                if (ik == 1) { const float c = __int_as_float(B.inv_value[q]); _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[q ? I1 : I0][t] = c; } \
                else if (ik == 2) { const int tsel = B.inv_value[q]; TADV_TEMP_SWITCH_ON(tsel, \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[q ? I1 : I0][t] = m.tmp[K][t];, \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[q ? I1 : I0][t] = spill[K][t];) } \
            } \
            int z = get_var(m.var, V); \
            const int lane = (int)(threadIdx.x & 31u); \
            const int dz = kind == BL_USUM ? UB : kind == BL_Z_LANE ? 32 * TA : 1; \
            const int hi = kind <= BL_USUM ? L.const_hi : loop_hi[a]; \
            const int lvl = L.mask_level; \
            const unsigned parent = kind == BL_SUM ? cur : kind == BL_USUM ? sum_parent : mstack[lvl - 1]; \
            /* per load slot: offset of this thread's element 0, its step per trip, pointer and element strides */ \
            unsigned xo[TADP_BODY_LOADS], xst[TADP_BODY_LOADS], xlc[TADP_BODY_LOADS], xuc[TADP_BODY_LOADS], xrs[REL ? TADP_BODY_LOADS : 1]; \
            const float *xbase[TADP_BODY_LOADS]; \
            _Pragma("unroll") for (int j = 0; j < TADP_BODY_LOADS; ++j) { \
                const TadpLoad &Ld = P.loads[B.load[j < B.n_loads ? j : 0]]; \
                xo[j] = load_offset(Ld, m.var); xst[j] = (unsigned)Ld.coef[V] * (unsigned)dz; \
                xlc[j] = (unsigned)Ld.lane_step; xuc[j] = UB > 1 ? (unsigned)Ld.unroll_step : 0u; \
                if (REL) xrs[j] = (unsigned)Ld.rel_step; \
                xbase[j] = ptrs.in[Ld.ptr]; \
            } \
            const uint2 steps = *reinterpret_cast<const uint2 *>(B.steps); \
            const int term = B.term; \
            constexpr unsigned FULL = T >= 32 ? 0xffffffffu : ((1u << T) - 1u); \
            for (;;) { \
                if (cur == FULL) TADV_XTRIP(SUMMODE, true) else TADV_XTRIP(SUMMODE, false) \
                z += dz; \
                const int zb = kind == BL_Z_LANE ? z - lane : z; \
                if (zb > hi) break; \
                _Pragma("unroll") for (int j = 0; j < TADP_BODY_LOADS; ++j) xo[j] += xst[j]; \
                if (kind == BL_Z_MASKED) { \
                    unsigned mk = 0; \
                    _Pragma("unroll") for (int t = 0; t < T; ++t) if (elo[lvl - 1][t] <= z && z <= ehi[lvl - 1][t]) mk |= 1u << t; \
                    cur = parent & mk; \
                } else if (zb + dz - 1 > hi) {   /* last trip of a loop that advances by more than one */ \
                    unsigned mk = 0; \
                    if (kind == BL_USUM) { _Pragma("unroll") for (int t = 0; t < T; ++t) if (z + (t % UB) <= hi) mk |= 1u << t; } \
                    else { _Pragma("unroll") for (int t = 0; t < T; ++t) if (z + 32 * (t / UB) <= hi) mk |= 1u << t; } \
                    cur = parent & mk; \
                } \
            } \
            cur = parent; \
        } break;
        TADV_XLOOP(0)
        TADV_XLOOP(1)

        default: {
            const int op = (raw.x & 0xffffu) >> 3;
            if (op == P_ZLOOP) TADV_ZLOOP_BODY
            else if (op == P_ZEND) TADV_ZEND_BODY
        } break;
        }
    }
}

}  // namespace tadvm

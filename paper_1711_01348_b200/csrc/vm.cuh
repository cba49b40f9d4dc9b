// Warp-uniform bytecode interpreter.
//
// One warp runs one work item at a time: the outer variables of the item are decoded from the
// item number, the lane variable is spread over the 32 lanes and over T vector elements per
// lane (element t of lane l has coordinate base + l + 32 t, so that every vector element of a
// load is one fully coalesced warp transaction).  All control flow (program counter, loop
// trip counts) is uniform across the warp; per-element validity is a T-bit activity mask.
//
// The operand stack is a register array indexed only by compile-time constants: the host
// encodes the stack depth into the handler number of every instruction, so each handler
// names its operands statically and nothing of the stack spills to local memory.
#pragma once
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "program.h"

namespace tadvm {

constexpr int WARPS_PER_BLOCK = 8;
constexpr int STACK = TADP_MAX_DEPTH - 1;   // usable depth (handlers are encoded for depth 0..7)

__device__ __forceinline__ int floor_div_i(int a, int b) { int q = a / b; return (a % b != 0 && a < 0) ? q - 1 : q; }
__device__ __forceinline__ int ceil_div_i(int a, int b) { int q = a / b; return (a % b != 0 && a > 0) ? q + 1 : q; }

__device__ __forceinline__ float powi_f(float x, int n)
{
    unsigned m = n < 0 ? (unsigned)(-n) : (unsigned)n;
    float r = 1.f, b = x;
    while (m) { if (m & 1u) r *= b; b *= b; m >>= 1; }
    return n < 0 ? 1.f / r : r;
}

template <int T>
struct Vm {
    float s[STACK][T];
    float tmp[TADP_NUM_TEMPS][T];
    float acc[T];
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

#define TADV_PUSHES(M, OP) M(OP, 0) M(OP, 1) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6)
#define TADV_FROM1(M, OP) M(OP, 1) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_FROM2(M, OP) M(OP, 2) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_FROM3(M, OP) M(OP, 3) M(OP, 4) M(OP, 5) M(OP, 6) M(OP, 7)
#define TADV_H(OP, D) ((OP) * TADP_MAX_DEPTH + (D))

// Runs the program of one work item.  mask0: which vector elements of this lane are live at
// the outermost level.  Returns in live_out the elements that accumulated at least one term.
template <int T, bool DEBUG>
__device__ __forceinline__ void run_item(const TadpProgram &P, const TadpPointers &ptrs, Vm<T> &m,
                                         unsigned mask0, unsigned &live_out)
{
    const int lane_var = P.lane_var;
    unsigned cur = mask0;                 // activity mask of the vector elements at the current loop level
    unsigned long long masks = mask0;     // byte k: mask at mask level k
    unsigned live = 0;
    int loop_hi[TADP_MAX_LOOPS];
    int elo[TADP_MAX_ZLOOPS][T], ehi[TADP_MAX_ZLOOPS][T];
    float spill[TADP_MAX_SPILL][T];
#pragma unroll
    for (int t = 0; t < T; ++t) m.acc[t] = 0.f;

    int pc = 0;
    for (;;) {
        const TadpInsn w = P.code[pc];
        ++pc;
        const int a = w.a;
        const int imm = w.imm;
        switch (w.handler) {
        case TADV_H(P_END, 0):
            live_out = live;
            return;

#define TADV_CONST(OP, D) case TADV_H(OP, D): { const float c = __int_as_float(imm); _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = c; } break;
        TADV_PUSHES(TADV_CONST, P_CONST)
#define TADV_ZERO(OP, D) case TADV_H(OP, D): { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = 0.f; } break;
        TADV_PUSHES(TADV_ZERO, P_ZERO)

#define TADV_LOAD(OP, D) case TADV_H(OP, D): { \
            const TadpLoad &L = P.loads[a]; \
            unsigned off = (unsigned)L.base; \
            _Pragma("unroll") for (int k = 0; k < TADP_MAX_VARS; ++k) off += (unsigned)L.coef[k] * (unsigned)m.var[k]; \
            const unsigned lc = (unsigned)L.coef[lane_var] * 32u; \
            const float *base = ptrs.in[L.ptr]; \
            _Pragma("unroll") for (int t = 0; t < T; ++t) { \
                const unsigned idx = off + (unsigned)t * lc; \
                bool ok = (cur >> t) & 1u; \
                if (DEBUG && ok && idx >= (unsigned)L.limit) { ok = false; if (ptrs.debug) atomicCAS(ptrs.debug, 0, 0x10000 + a); } \
                m.s[D][t] = ok ? __ldg(base + idx) : 0.f; \
            } } break;
        TADV_PUSHES(TADV_LOAD, P_LOAD)

#define TADV_UNARY(D, EXPR) { _Pragma("unroll") for (int t = 0; t < T; ++t) { const float x = m.s[D - 1][t]; m.s[D - 1][t] = (EXPR); } } break;
#define TADV_NEG(OP, D) case TADV_H(OP, D): TADV_UNARY(D, -x)
        TADV_FROM1(TADV_NEG, P_NEG)
#define TADV_EXP(OP, D) case TADV_H(OP, D): TADV_UNARY(D, expf(x))
        TADV_FROM1(TADV_EXP, P_EXP)
#define TADV_LOG(OP, D) case TADV_H(OP, D): TADV_UNARY(D, logf(x))
        TADV_FROM1(TADV_LOG, P_LOG)
#define TADV_SIN(OP, D) case TADV_H(OP, D): TADV_UNARY(D, sinf(x))
        TADV_FROM1(TADV_SIN, P_SIN)
#define TADV_COS(OP, D) case TADV_H(OP, D): TADV_UNARY(D, cosf(x))
        TADV_FROM1(TADV_COS, P_COS)
#define TADV_TANH(OP, D) case TADV_H(OP, D): TADV_UNARY(D, tanhf(x))
        TADV_FROM1(TADV_TANH, P_TANH)
#define TADV_SINH(OP, D) case TADV_H(OP, D): TADV_UNARY(D, sinhf(x))
        TADV_FROM1(TADV_SINH, P_SINH)
#define TADV_COSH(OP, D) case TADV_H(OP, D): TADV_UNARY(D, coshf(x))
        TADV_FROM1(TADV_COSH, P_COSH)
#define TADV_SQR(OP, D) case TADV_H(OP, D): TADV_UNARY(D, x * x)
        TADV_FROM1(TADV_SQR, P_SQR)
#define TADV_POWI(OP, D) case TADV_H(OP, D): TADV_UNARY(D, powi_f(x, imm))
        TADV_FROM1(TADV_POWI, P_POWI)
#define TADV_MULC(OP, D) case TADV_H(OP, D): { const float c = __int_as_float(imm); TADV_UNARY(D, x * c) }
        TADV_FROM1(TADV_MULC, P_MULC)
#define TADV_ADDC(OP, D) case TADV_H(OP, D): { const float c = __int_as_float(imm); TADV_UNARY(D, x + c) }
        TADV_FROM1(TADV_ADDC, P_ADDC)

#define TADV_BINARY(D, EXPR) { _Pragma("unroll") for (int t = 0; t < T; ++t) { const float x = m.s[D - 2][t], y = m.s[D - 1][t]; m.s[D - 2][t] = (EXPR); } } break;
#define TADV_ADD(OP, D) case TADV_H(OP, D): TADV_BINARY(D, x + y)
        TADV_FROM2(TADV_ADD, P_ADD)
        TADV_FROM2(TADV_ADD, P_SUMADD)
#define TADV_SUB(OP, D) case TADV_H(OP, D): TADV_BINARY(D, x - y)
        TADV_FROM2(TADV_SUB, P_SUB)
#define TADV_MUL(OP, D) case TADV_H(OP, D): TADV_BINARY(D, x * y)
        TADV_FROM2(TADV_MUL, P_MUL)
#define TADV_DIV(OP, D) case TADV_H(OP, D): TADV_BINARY(D, x / y)
        TADV_FROM2(TADV_DIV, P_DIV)
#define TADV_FMA(OP, D) case TADV_H(OP, D): { _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D - 3][t] = fmaf(m.s[D - 3][t], m.s[D - 2][t], m.s[D - 1][t]); } break;
        TADV_FROM3(TADV_FMA, P_FMA)

#define TADV_TEMP_SWITCH(STMT_REG, STMT_SPILL) \
            switch (a) { \
            case 0: { constexpr int K = 0; STMT_REG } break; case 1: { constexpr int K = 1; STMT_REG } break; \
            case 2: { constexpr int K = 2; STMT_REG } break; case 3: { constexpr int K = 3; STMT_REG } break; \
            case 4: { constexpr int K = 4; STMT_REG } break; case 5: { constexpr int K = 5; STMT_REG } break; \
            case 6: { constexpr int K = 6; STMT_REG } break; case 7: { constexpr int K = 7; STMT_REG } break; \
            default: { const int K = a - TADP_NUM_TEMPS; STMT_SPILL } break; }
#define TADV_LDT(OP, D) case TADV_H(OP, D): { TADV_TEMP_SWITCH( \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = m.tmp[K][t];, \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.s[D][t] = spill[K][t];) } break;
        TADV_PUSHES(TADV_LDT, P_LDT)
#define TADV_STT(OP, D) case TADV_H(OP, D): { TADV_TEMP_SWITCH( \
            _Pragma("unroll") for (int t = 0; t < T; ++t) m.tmp[K][t] = m.s[D - 1][t];, \
            _Pragma("unroll") for (int t = 0; t < T; ++t) spill[K][t] = m.s[D - 1][t];) } break;
        TADV_FROM1(TADV_STT, P_STT)

#define TADV_ACC(OP, D) case TADV_H(OP, D): { _Pragma("unroll") for (int t = 0; t < T; ++t) if ((cur >> t) & 1u) m.acc[t] += m.s[D - 1][t]; live |= cur; } break;
        TADV_FROM1(TADV_ACC, P_ACC)

        default: {
            // loop control: handlers of every depth share one body (the stack is not touched)
            const int op = w.handler / TADP_MAX_DEPTH;
            const TadpLoop &L = P.loops[a];
            if (op == P_SLOOP) {
                if (L.const_lo > L.const_hi) pc = imm;
                else set_var(m.var, L.var, L.const_lo);
            } else if (op == P_SEND) {
                const int k = get_var(m.var, L.var) + 1;
                if (k <= L.const_hi) { set_var(m.var, L.var, k); pc = imm; }
            } else if (op == P_ZLOOP) {
                const int lvl = L.mask_level;
                const unsigned parent = (unsigned)(masks >> (8 * (lvl - 1))) & 0xffu;
                int wlo, whi;
                if (L.is_lane || !L.depends_on_lane) {
                    // bounds are the same for the whole warp
                    int lo = INT_MIN, hi = INT_MAX;
                    for (int r = 0; r < L.n_lower; ++r) { const TadpRow &R = P.rows[L.lower0 + r]; const int nmr = row_num(R, m.var); lo = max(lo, R.den == 1 ? nmr : ceil_div_i(nmr, R.den)); }
                    for (int r = 0; r < L.n_upper; ++r) { const TadpRow &R = P.rows[L.upper0 + r]; const int nmr = row_num(R, m.var); hi = min(hi, R.den == 1 ? nmr : floor_div_i(nmr, R.den)); }
                    wlo = lo; whi = hi;
                    if (__ballot_sync(0xffffffffu, parent != 0) == 0) { wlo = 1; whi = 0; }   // nothing live in the warp
                } else {
                    int lo_w = INT_MAX, hi_w = INT_MIN;
#pragma unroll
                    for (int t = 0; t < T; ++t) { elo[lvl - 1][t] = INT_MIN; ehi[lvl - 1][t] = INT_MAX; }
                    for (int r = 0; r < L.n_lower; ++r) {
                        const TadpRow &R = P.rows[L.lower0 + r];
                        const int nmr = row_num(R, m.var); const int step = R.coef[lane_var] * 32;
#pragma unroll
                        for (int t = 0; t < T; ++t) { int v = nmr + t * step; v = R.den == 1 ? v : ceil_div_i(v, R.den); elo[lvl - 1][t] = max(elo[lvl - 1][t], v); }
                    }
                    for (int r = 0; r < L.n_upper; ++r) {
                        const TadpRow &R = P.rows[L.upper0 + r];
                        const int nmr = row_num(R, m.var); const int step = R.coef[lane_var] * 32;
#pragma unroll
                        for (int t = 0; t < T; ++t) { int v = nmr + t * step; v = R.den == 1 ? v : floor_div_i(v, R.den); ehi[lvl - 1][t] = min(ehi[lvl - 1][t], v); }
                    }
#pragma unroll
                    for (int t = 0; t < T; ++t)
                        if (((parent >> t) & 1u) && elo[lvl - 1][t] <= ehi[lvl - 1][t]) { lo_w = min(lo_w, elo[lvl - 1][t]); hi_w = max(hi_w, ehi[lvl - 1][t]); }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) { lo_w = min(lo_w, __shfl_xor_sync(0xffffffffu, lo_w, o)); hi_w = max(hi_w, __shfl_xor_sync(0xffffffffu, hi_w, o)); }
                    wlo = lo_w; whi = hi_w;
                }
                if (wlo > whi) { pc = imm; }
                else {
                    loop_hi[a] = whi;
                    unsigned mk;
                    if (L.is_lane) {
                        const int z = wlo + (int)(threadIdx.x & 31u);
                        set_var(m.var, L.var, z);
                        mk = 0;
#pragma unroll
                        for (int t = 0; t < T; ++t) if (z + 32 * t <= whi) mk |= 1u << t;
                        mk &= parent;
                    } else {
                        set_var(m.var, L.var, wlo);
                        mk = parent;
                        if (L.depends_on_lane) {
                            mk = 0;
#pragma unroll
                            for (int t = 0; t < T; ++t) if (elo[lvl - 1][t] <= wlo && wlo <= ehi[lvl - 1][t]) mk |= 1u << t;
                            mk &= parent;
                        }
                    }
                    cur = mk;
                    masks = (masks & ~(0xffull << (8 * lvl))) | ((unsigned long long)mk << (8 * lvl));
                }
            } else if (op == P_ZEND) {
                const int lvl = L.mask_level;
                const unsigned parent = (unsigned)(masks >> (8 * (lvl - 1))) & 0xffu;
                const int whi = loop_hi[a];
                const int z = get_var(m.var, L.var) + (L.is_lane ? 32 * T : 1);
                const int zbase = L.is_lane ? z - (int)(threadIdx.x & 31u) : z;
                if (zbase <= whi) {
                    set_var(m.var, L.var, z);
                    unsigned mk;
                    if (L.is_lane) {
                        mk = 0;
#pragma unroll
                        for (int t = 0; t < T; ++t) if (z + 32 * t <= whi) mk |= 1u << t;
                        mk &= parent;
                    } else if (L.depends_on_lane) {
                        mk = 0;
#pragma unroll
                        for (int t = 0; t < T; ++t) if (elo[lvl - 1][t] <= z && z <= ehi[lvl - 1][t]) mk |= 1u << t;
                        mk &= parent;
                    } else mk = parent;
                    cur = mk;
                    masks = (masks & ~(0xffull << (8 * lvl))) | ((unsigned long long)mk << (8 * lvl));
                    pc = imm;
                } else {
                    cur = parent;
                }
            }
        } break;
        }
    }
}

}  // namespace tadvm

// Tile kernel for contraction programs (contract.h): a thread block owns a BM x BN tile of
// outputs, gathers BK summation indices of both operands at a time into shared memory with
// asynchronous copies (two stages), and every thread keeps a TM x TN tile of sums in
// registers that it feeds from shared memory with 128-bit loads.  Operand elements outside a
// guard, past the end of the summation range or in the ragged edge of a tile arrive as zeros
// (zero-fill copies), so the multiply-add loop has no tests.  No atomics: a summation split over
// several blocks writes planes of partial sums that tad_contract_reduce adds in a fixed order.
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>

#include "contract.h"
#include "program.h"

namespace {

constexpr int BK = TADC_BK;
constexpr int KK_UNROLL = 8;          // summation indices per unrolled body of the multiply-add loop
constexpr int STAGES = 2;
constexpr int DEAD = INT_MIN / 2;      // guard part of a row or summation index that does not exist

__device__ __forceinline__ void cp_async4(float *dst, const float *src, bool live)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst);
    const int bytes = live ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(d), "l"(src), "r"(bytes));
}
__device__ __forceinline__ void cp_async16(float *dst, const float *src, bool live)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(dst);
    const int bytes = live ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(src), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

struct Parts { int a, b, o, ga, gb; };

// digits of a flattened index, last digit fastest, folded into the offset parts of the group
__device__ __forceinline__ Parts decode(const TadcGroup &G, unsigned idx)
{
    Parts p{0, 0, 0, 0, 0};
#pragma unroll
    for (int d = TADC_MAX_DIGITS - 1; d >= 0; --d) {
        if (d < G.n_digits) {
            const unsigned e = (unsigned)G.ext[d];
            const unsigned q = idx / e;
            const int r = (int)(idx - q * e);
            idx = q;
            p.a += r * G.sA[d]; p.b += r * G.sB[d]; p.o += r * G.sO[d];
            p.ga += r * G.gA[d]; p.gb += r * G.gB[d];
        }
    }
    return p;
}

// One stage of one operand: BK x BR values into smem[kl * (BR + 4) + rl].  rows[rl] = (offset part, guard
// part) of tile row rl, ktab[kl] the same for the stage's summation index kl.  CHECK = false is the path
// of a stage whose every element exists and is read (no guard on the operand, tile and stage inside
// the ranges): offset add, copy.  pre = rows[row of this thread] for the modes whose threads keep one row.
template <int BR, int NT, bool CHECK>
__device__ __forceinline__ void gather(float *smem, const float *__restrict__ src, const int2 *rows, const int2 *ktab,
                                       const int2 pre, const int mode, const unsigned gext, const unsigned tid, const unsigned klimit)
{
    // The copies carry no memory clobber (the group commit and wait do), and the table entries of a batch of
    // copies are read before the first of them is issued, so that the table reads overlap instead of each
    // waiting its turn.  klimit: summation indices of this stage that the multiply-add loop will read.
    constexpr int LD = BR + 4;
    constexpr bool REGULAR = NT % BR == 0 && (BR * BK) % NT == 0 && NT % (BR / 4) == 0 && NT % (4 * BK) == 0;
    if constexpr (!REGULAR) {
        // any number of threads: element e of the stage -> (row, summation index) by the mode's own order
        const unsigned total = mode == TG_ROW16 ? (BR / 4) * BK : BR * BK;
        for (unsigned e0 = tid; e0 < total; e0 += 4 * NT) {
            unsigned off[4], dst[4]; bool live[4], use[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned e = e0 + j * NT;
                unsigned rl, kl;
                if (mode == TG_ROW16) { rl = (e % (BR / 4)) * 4; kl = e / (BR / 4); }
                else if (mode == TG_ROW) { rl = e % BR; kl = e / BR; }
                else { kl = e % BK; rl = e / BK; }
                use[j] = e < total && kl < klimit;
                const int2 r = rows[use[j] ? rl : 0], kt = ktab[use[j] ? kl : 0];
                live[j] = !CHECK || (unsigned)(r.y + kt.y) < gext;
                off[j] = live[j] ? (unsigned)(r.x + kt.x) : 0u;
                dst[j] = kl * LD + rl;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (use[j]) { if (mode == TG_ROW16) cp_async16(smem + dst[j], src + off[j], live[j]); else cp_async4(smem + dst[j], src + off[j], live[j]); }
        }
        return;
    } else {
    if (mode == TG_ROW16) {
        constexpr unsigned CH = BR / 4, TOTAL = CH * BK, PER = (TOTAL + NT - 1) / NT, KSTEP = NT / CH;
        const unsigned rl = (tid % CH) * 4, kl0 = tid / CH;
        if (TOTAL % NT != 0 && kl0 >= BK) return;
        unsigned off[PER]; bool live[PER];
#pragma unroll
        for (unsigned j = 0; j < PER; ++j) {
            const int2 kt = ktab[kl0 + KSTEP * j];
            live[j] = !CHECK || (unsigned)(pre.y + kt.y) < gext;
            off[j] = live[j] ? (unsigned)(pre.x + kt.x) : 0u;
        }
#pragma unroll
        for (unsigned j = 0; j < PER; ++j)
            if (kl0 + KSTEP * j < klimit) cp_async16(smem + (kl0 + KSTEP * j) * LD + rl, src + off[j], live[j]);
    } else if (mode == TG_ROW) {
        constexpr unsigned TOTAL = BR * BK, PER = TOTAL / NT, KSTEP = NT / BR;
        const unsigned rl = tid % BR, kl0 = tid / BR;
        unsigned off[PER]; bool live[PER];
#pragma unroll
        for (unsigned j = 0; j < PER; ++j) {
            const int2 kt = ktab[kl0 + KSTEP * j];
            live[j] = !CHECK || (unsigned)(pre.y + kt.y) < gext;
            off[j] = live[j] ? (unsigned)(pre.x + kt.x) : 0u;
        }
#pragma unroll
        for (unsigned j = 0; j < PER; ++j)
            if (kl0 + KSTEP * j < klimit) cp_async4(smem + (kl0 + KSTEP * j) * LD + rl, src + off[j], live[j]);
    } else {
        // a warp copies 8 summation indices x 4 rows: full 32-byte sectors of a row-major operand, and the
        // 32 shared-memory words it writes (row stride BR + 4) fall into 32 different banks
        constexpr unsigned TOTAL = BR * BK, PER = TOTAL / NT, RSTEP = NT / BK;
        const unsigned kl = (tid % 8) + 8 * ((tid / 32) % (BK / 8)), rl0 = (tid / 8) % 4 + 4 * (tid / (4 * BK));
        if (kl >= klimit) return;
        const int2 kt = ktab[kl];
        unsigned off[PER]; bool live[PER];
#pragma unroll
        for (unsigned j = 0; j < PER; ++j) {
            const int2 r = rows[rl0 + RSTEP * j];
            live[j] = !CHECK || (unsigned)(r.y + kt.y) < gext;
            off[j] = live[j] ? (unsigned)(r.x + kt.x) : 0u;
        }
#pragma unroll
        for (unsigned j = 0; j < PER; ++j) cp_async4(smem + kl * LD + rl0 + RSTEP * j, src + off[j], live[j]);
    }
    }
}

__device__ __forceinline__ float own_tanh(float x)
{
    const float ax = fabsf(x);
    const float e = __expf(2.f * ax);
    const float t = 1.f - __fdividef(2.f, e + 1.f);
    const float x2 = x * x;
    const float small = x * (1.f + x2 * (-0.33333334f + x2 * (0.13333334f + x2 * -0.05396825f)));
    return ax < 0.25f ? small : copysignf(t, x);
}

// the steps every finished sum goes through before it is stored
__device__ __forceinline__ float epilogue(const TadcProgram &P, const TadpPointers &ptrs, float v, unsigned off)
{
    for (int s = 0; s < P.n_epi; ++s) {
        switch (P.epi_op[s]) {
        case TE_NEG: v = -v; break;
        case TE_EXP: v = __expf(v); break;
        case TE_MULC: v *= P.epi_imm[s]; break;
        case TE_ADDC: v += P.epi_imm[s]; break;
        case TE_SQR: v *= v; break;
        case TE_TANH: v = own_tanh(v); break;
        case TE_MUL_LOAD: v *= __ldg(ptrs.in[P.epi_ptr[s]] + (unsigned)(P.epi_base[s] + (int)off)); break;
        case TE_ADD_LOAD: v += __ldg(ptrs.in[P.epi_ptr[s]] + (unsigned)(P.epi_base[s] + (int)off)); break;
        default: break;
        }
    }
    return v;
}

template <int BM, int BN, int TM, int TN>
struct Cfg {
    static constexpr int NT = (BM / TM) * (BN / TN);
    static constexpr int LDA = BM + 4, LDB = BN + 4;
    static constexpr int STAGE_FLOATS = BK * (LDA + LDB);
    static constexpr size_t SMEM = size_t(STAGES) * STAGE_FLOATS * 4 + size_t(BM + BN) * 8 + size_t(BM + BN) * 4 +
                                   size_t(STAGES + 1) * BK * 16;      // stages, row tables, output offsets, two k tables
};

template <int BM, int BN, int TM, int TN>
__global__ void __launch_bounds__(Cfg<BM, BN, TM, TN>::NT, (TM * TN >= 64 ? 2 : Cfg<BM, BN, TM, TN>::NT <= 160 ? 4 : 3))
tad_contract_kernel(const __grid_constant__ TadcProgram P, const __grid_constant__ TadpPointers ptrs, const unsigned tiles_m, const unsigned tiles_n)
{
    using C = Cfg<BM, BN, TM, TN>;
    constexpr int NT = C::NT, LDA = C::LDA, LDB = C::LDB;
    constexpr int GM = TM / 4, GN = TN / 4;           // groups of four rows / columns per thread
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *stage_mem = reinterpret_cast<float *>(smem_raw);
    int2 *ktabA = reinterpret_cast<int2 *>(stage_mem + STAGES * C::STAGE_FLOATS);
    int2 *ktabB = ktabA + (STAGES + 1) * BK;
    int2 *rowA = ktabB + (STAGES + 1) * BK;
    int2 *rowB = rowA + BM;
    int *outM = reinterpret_cast<int *>(rowB + BN);
    int *outN = outM + BM;

    const unsigned tid = threadIdx.x;
    const unsigned tile = blockIdx.x;
    const unsigned tile_m = tile % tiles_m, tile_n = tile / tiles_m;
    const unsigned ks = blockIdx.y, zb = blockIdx.z;
    const Parts z = decode(P.Z, zb);
    // Offsets are sums of signed 32-bit parts that may be negative one by one (a band that starts below
    // zero, a negative stride); only the complete sum of a live element is a valid element offset, so the
    // constant parts go into the row tables and the pointer stays the tensor's own.
    const bool onesB = P.ptrB < 0;                // B is a tensor of ones: a plain summation of A
    const float *__restrict__ A = ptrs.in[P.ptrA];
    const float *__restrict__ B = onesB ? A : ptrs.in[P.ptrB];
    const int constA = P.baseA + z.a, constB = P.baseB + z.b;
    const unsigned Mext = (unsigned)P.M.extent, Next = (unsigned)P.N.extent;
    const unsigned kbeg = ks * (unsigned)P.kchunk;
    const unsigned kend = min((unsigned)P.K.extent, kbeg + (unsigned)P.kchunk);
    const int n_stages = (int)((kend - kbeg + BK - 1) / BK);

    // per-row parts of the operand offsets, guards and output offsets of this tile
    for (unsigned r = tid; r < BM; r += NT) {
        const unsigned m = tile_m * BM + r;
        if (m < Mext) { const Parts p = decode(P.M, m); rowA[r] = make_int2(constA + p.a, P.guardA_c0 + z.ga + p.ga); outM[r] = p.o; }
        else { rowA[r] = make_int2(0, DEAD); outM[r] = 0; }
    }
    for (unsigned r = tid; r < BN; r += NT) {
        const unsigned n = tile_n * BN + r;
        if (n < Next) { const Parts p = decode(P.N, n); rowB[r] = make_int2(constB + p.b, P.guardB_c0 + z.gb + p.gb); outN[r] = p.o; }
        else { rowB[r] = make_int2(0, DEAD); outN[r] = 0; }
    }
    auto fill_ktab = [&](int kstage) {
        if (tid < BK) {
            const unsigned k = kbeg + (unsigned)kstage * BK + tid;
            int2 ea = make_int2(0, DEAD), eb = make_int2(0, DEAD);
            if (k < kend) { const Parts p = decode(P.K, k); ea = make_int2(p.a, p.ga); eb = make_int2(p.b, p.gb); }
            ktabA[(kstage % (STAGES + 1)) * BK + tid] = ea;
            ktabB[(kstage % (STAGES + 1)) * BK + tid] = eb;
        }
    };
    for (int s = 0; s < STAGES; ++s) fill_ktab(s);
    if (onesB)
        for (unsigned e = tid; e < (unsigned)(STAGES * BK * LDB); e += NT) {
            const unsigned s = e / (BK * LDB), r = e - s * (BK * LDB);
            stage_mem[s * C::STAGE_FLOATS + BK * LDA + r] = 1.f;
        }
    __syncthreads();
    const unsigned gextA = (unsigned)P.guardA_ext, gextB = (unsigned)P.guardB_ext;
    const int modeA = P.modeA, modeB = P.modeB;
    // the row a thread keeps through all stages (modes with the lanes along the row index)
    const int2 preA = rowA[modeA == TG_ROW16 ? (tid % (BM / 4)) * 4 : tid % BM];
    const int2 preB = rowB[modeB == TG_ROW16 ? (tid % (BN / 4)) * 4 : tid % BN];      // (unused by tiles with irregular thread counts)
    // tiles inside the ranges and operands without a guard take the copy path without tests
    const bool plainA = !P.guardA && (tile_m + 1) * BM <= Mext, plainB = !P.guardB && (tile_n + 1) * BN <= Next;
    auto issue = [&](int kstage) {
        if (kstage < n_stages) {
            float *as = stage_mem + (kstage % STAGES) * C::STAGE_FLOATS;
            float *bs = as + BK * LDA;
            const int slot = (kstage % (STAGES + 1)) * BK;
            const unsigned left = kend - kbeg - (unsigned)kstage * BK;
            const bool full = left >= BK;
            const unsigned klimit = full ? BK : (left + KK_UNROLL - 1) / KK_UNROLL * KK_UNROLL;
            if (plainA && full) gather<BM, NT, false>(as, A, rowA, ktabA + slot, preA, modeA, gextA, tid, klimit);
            else gather<BM, NT, true>(as, A, rowA, ktabA + slot, preA, modeA, gextA, tid, klimit);
            if (onesB) {}
            else if (plainB && full) gather<BN, NT, false>(bs, B, rowB, ktabB + slot, preB, modeB, gextB, tid, klimit);
            else gather<BN, NT, true>(bs, B, rowB, ktabB + slot, preB, modeB, gextB, tid, klimit);
        }
        cp_async_commit();
    };
    for (int s = 0; s < STAGES - 1; ++s) issue(s);

    // a warp covers 8 thread columns x 4 thread rows: its 128-bit reads of a stage touch 128 consecutive bytes
    // of the B tile and 64 of the A tile, one shared-memory wavefront each (tiles whose thread columns do not
    // come in eights number their threads row by row)
    constexpr unsigned TCOLS = BN / TN;
    const unsigned warp = tid / 32, lane = tid % 32;
    const int tx = TCOLS % 8 == 0 ? (int)((warp % (TCOLS / 8 ? TCOLS / 8 : 1)) * 8 + lane % 8) : (int)(tid % TCOLS);
    const int ty = TCOLS % 8 == 0 ? (int)((warp / (TCOLS / 8 ? TCOLS / 8 : 1)) * 4 + lane / 8) : (int)(tid / TCOLS);
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    for (int it = 0; it < n_stages; ++it) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        fill_ktab(it + STAGES);
        issue(it + STAGES - 1);
        const float *as = stage_mem + (it % STAGES) * C::STAGE_FLOATS;
        const float *bs = as + BK * LDA;
        // operands of summation index kk + 1 are fetched from shared memory while those of kk are multiplied
        float a[2][TM], b[2][TN];
        auto fetch = [&](int kk, float *av, float *bv) {
#pragma unroll
            for (int g = 0; g < GM; ++g) {
                const float4 v = *reinterpret_cast<const float4 *>(as + kk * LDA + g * (BM / GM) + ty * 4);
                av[4 * g] = v.x; av[4 * g + 1] = v.y; av[4 * g + 2] = v.z; av[4 * g + 3] = v.w;
            }
#pragma unroll
            for (int g = 0; g < GN; ++g) {
                const float4 v = *reinterpret_cast<const float4 *>(bs + kk * LDB + g * (BN / GN) + tx * 4);
                bv[4 * g] = v.x; bv[4 * g + 1] = v.y; bv[4 * g + 2] = v.z; bv[4 * g + 3] = v.w;
            }
        };
        fetch(0, a[0], b[0]);
        // bodies of KK_UNROLL summation indices; a last stage with few indices left runs only the bodies that hold some
        const int n_bodies = min(BK / KK_UNROLL, (int)(((kend - kbeg) - (unsigned)it * BK + KK_UNROLL - 1) / KK_UNROLL));
        for (int body = 0; body < n_bodies; ++body) {
            const float *as_b = as + body * KK_UNROLL * LDA, *bs_b = bs + body * KK_UNROLL * LDB;
#pragma unroll
            for (int u = 0; u < KK_UNROLL; ++u) {
                if (u + 1 < KK_UNROLL || body + 1 < n_bodies) {
#pragma unroll
                    for (int q = 0; q < GM; ++q) {
                        const float4 v = *reinterpret_cast<const float4 *>(as_b + (u + 1) * LDA + q * (BM / GM) + ty * 4);
                        a[(u + 1) & 1][4 * q] = v.x; a[(u + 1) & 1][4 * q + 1] = v.y; a[(u + 1) & 1][4 * q + 2] = v.z; a[(u + 1) & 1][4 * q + 3] = v.w;
                    }
#pragma unroll
                    for (int q = 0; q < GN; ++q) {
                        const float4 v = *reinterpret_cast<const float4 *>(bs_b + (u + 1) * LDB + q * (BN / GN) + tx * 4);
                        b[(u + 1) & 1][4 * q] = v.x; b[(u + 1) & 1][4 * q + 1] = v.y; b[(u + 1) & 1][4 * q + 2] = v.z; b[(u + 1) & 1][4 * q + 3] = v.w;
                    }
                }
#pragma unroll
                for (int i = 0; i < TM; ++i)
#pragma unroll
                    for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[u & 1][i], b[u & 1][j], acc[i][j]);
            }
        }
    }
    cp_async_wait<0>();

    // ---- store ----
    // The sums go through shared memory (the stage buffers are free now): a compact loop then applies the epilogue
    // to four columns at a time and writes whole rows of the tile, consecutive threads to consecutive columns.
    // (Storing straight from the 64 registers would unroll the epilogue 64 times: code that no longer fits the
    // instruction cache and is run once per tile.)
    constexpr int LDC = BN + 4;
    static_assert(BM * LDC <= STAGES * C::STAGE_FLOATS, "the tile of sums must fit into the stage buffers");
    float *cs = stage_mem;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int rl = (i / 4) * (BM / GM) + ty * 4 + (i % 4);
#pragma unroll
        for (int q = 0; q < GN; ++q)
            *reinterpret_cast<float4 *>(cs + rl * LDC + q * (BN / GN) + tx * 4) =
                make_float4(acc[i][4 * q], acc[i][4 * q + 1], acc[i][4 * q + 2], acc[i][4 * q + 3]);
    }
    __syncthreads();
    const bool partial = P.ksplit > 1;
    float *__restrict__ out = partial ? ptrs.part : ptrs.out;
    const float scale = P.scale;
    const int n_epi = partial ? 0 : P.n_epi;
    const int obase = P.baseO + z.o;
    const bool vec_ok = partial ? (Next & 3u) == 0 : P.out_vec4 != 0;
    // four pieces of four columns per pass: every epilogue step is dispatched once for 16 values and the loads of a
    // step (a tensor laid out like the output) are issued together
    constexpr int EU = 4;
    for (unsigned e0 = tid; e0 < (unsigned)(BM * BN / 4); e0 += NT * EU) {
        float v[EU][4];
        unsigned off[EU][4];
        int live[EU];
#pragma unroll
        for (int u = 0; u < EU; ++u) {
            const unsigned e = e0 + (unsigned)u * NT;
            const unsigned rl = e / (BN / 4), cl = (e % (BN / 4)) * 4;
            const unsigned m = tile_m * BM + rl, n = tile_n * BN + cl;
            const bool in = e < (unsigned)(BM * BN / 4) && m < Mext && n < Next;
            live[u] = in ? (int)min(4u, Next - n) : 0;
            const float4 s4 = in ? *reinterpret_cast<const float4 *>(cs + rl * LDC + cl) : make_float4(0.f, 0.f, 0.f, 0.f);
            v[u][0] = s4.x; v[u][1] = s4.y; v[u][2] = s4.z; v[u][3] = s4.w;
            if (partial) {
                const unsigned o0 = (unsigned)(((zb * (unsigned)P.ksplit + ks) * Mext + m) * Next + n);     // < 2^25 cells per plane set
#pragma unroll
                for (int j = 0; j < 4; ++j) off[u][j] = in ? o0 + j : 0u;
            } else {
                const int ob = obase + outM[in ? rl : 0];
                if (vec_ok) {
                    const unsigned o0 = (unsigned)(ob + outN[in ? cl : 0]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) { off[u][j] = o0 + j; v[u][j] *= scale; }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) { off[u][j] = (unsigned)(ob + outN[in && j < live[u] ? cl + j : 0]); v[u][j] *= scale; }
                }
            }
        }
#define TAD_EPI_ALL(expr)                                               \
    _Pragma("unroll") for (int u = 0; u < EU; ++u)                       \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) { expr; }
        for (int s = 0; s < n_epi; ++s) {
            const int op = P.epi_op[s];
            const float imm = P.epi_imm[s];
            const float *src = (op == TE_MUL_LOAD || op == TE_ADD_LOAD) ? ptrs.in[P.epi_ptr[s]] : nullptr;
            const int sb = P.epi_base[s];
            switch (op) {
            case TE_NEG: TAD_EPI_ALL(v[u][j] = -v[u][j]) break;
            case TE_EXP: TAD_EPI_ALL(v[u][j] = __expf(v[u][j])) break;
            case TE_MULC: TAD_EPI_ALL(v[u][j] *= imm) break;
            case TE_ADDC: TAD_EPI_ALL(v[u][j] += imm) break;
            case TE_SQR: TAD_EPI_ALL(v[u][j] *= v[u][j]) break;
            case TE_TANH: TAD_EPI_ALL(v[u][j] = own_tanh(v[u][j])) break;
            case TE_MUL_LOAD: case TE_ADD_LOAD: {
                float w[EU][4];
                if (vec_ok && ((sb & 3) == 0) && ((reinterpret_cast<uintptr_t>(src) & 15u) == 0)) {
#pragma unroll
                    for (int u = 0; u < EU; ++u) {
                        const float4 w4 = live[u] ? __ldg(reinterpret_cast<const float4 *>(src + (unsigned)(sb + (int)off[u][0]))) : make_float4(0.f, 0.f, 0.f, 0.f);
                        w[u][0] = w4.x; w[u][1] = w4.y; w[u][2] = w4.z; w[u][3] = w4.w;
                    }
                } else {
                    TAD_EPI_ALL(w[u][j] = j < live[u] ? __ldg(src + (unsigned)(sb + (int)off[u][j])) : 0.f)
                }
                if (op == TE_MUL_LOAD) { TAD_EPI_ALL(v[u][j] *= w[u][j]) } else { TAD_EPI_ALL(v[u][j] += w[u][j]) }
                break;
            }
            default: break;
            }
        }
#undef TAD_EPI_ALL
#pragma unroll
        for (int u = 0; u < EU; ++u) {
            if (!live[u]) continue;
            if (vec_ok) {
                float4 *dst = reinterpret_cast<float4 *>(out + off[u][0]);
                float4 r = make_float4(v[u][0], v[u][1], v[u][2], v[u][3]);
                if (!partial && P.accumulate) { const float4 o = *dst; r.x += o.x; r.y += o.y; r.z += o.z; r.w += o.w; }
                *dst = r;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < live[u]) out[off[u][j]] = (!partial && P.accumulate) ? v[u][j] + out[off[u][j]] : v[u][j];
            }
        }
    }
}

// Adds the planes of partial sums of a split summation, plane 0 first, and stores the outputs.
__global__ void __launch_bounds__(256)
tad_contract_reduce(const __grid_constant__ TadcProgram P, const __grid_constant__ TadpPointers ptrs)
{
    const unsigned Mext = (unsigned)P.M.extent, Next = (unsigned)P.N.extent;
    const unsigned per_z = Mext * Next;
    const unsigned cells = per_z * (unsigned)P.Z.extent;
    const unsigned planes = (unsigned)P.ksplit;
    for (unsigned c = blockIdx.x * blockDim.x + threadIdx.x; c < cells; c += gridDim.x * blockDim.x) {
        const unsigned zb = c / per_z, rem = c - zb * per_z;
        const unsigned m = rem / Next, n = rem - m * Next;
        const float *src = ptrs.part + (size_t)zb * planes * per_z + rem;
        float sum = 0.f;
        for (unsigned s = 0; s < planes; ++s) sum += src[(size_t)s * per_z];
        const unsigned off = (unsigned)(P.baseO + decode(P.Z, zb).o + decode(P.M, m).o + decode(P.N, n).o);
        float v = epilogue(P, ptrs, sum * P.scale, off);
        if (P.accumulate) v += ptrs.out[off];
        ptrs.out[off] = v;
    }
}

// Plain summation of one operand (contraction with a tensor of ones and a single output column):
//     out[m] (+)= scale * sum_k A[row(m) + k * stride]
// One warp per output; its lanes walk the summation index (128-bit loads when that index is contiguous
// and aligned), then a fixed-order shuffle tree.  Bound by HBM: every element of A is read once.
__global__ void __launch_bounds__(256)
tad_rowsum_kernel(const __grid_constant__ TadcProgram P, const __grid_constant__ TadpPointers ptrs)
{
    const unsigned lane = threadIdx.x & 31u;
    const unsigned warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = (gridDim.x * blockDim.x) >> 5;
    const float *__restrict__ A = ptrs.in[P.ptrA];
    const bool weighted = P.ptrB >= 0;                   // B[k]: one weight per summation index
    const float *__restrict__ B = weighted ? ptrs.in[P.ptrB] : A;
    const int kb = P.K.n_digits ? P.K.sB[0] : 0;
    const unsigned K = (unsigned)P.K.extent;
    const int ks = P.K.n_digits ? P.K.sA[0] : 0;
    for (unsigned m = warp; m < (unsigned)P.M.extent; m += n_warps) {
        const Parts p = decode(P.M, m);
        const int base = P.baseA + p.a;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        if (weighted && ks == 1 && kb == 1 && ((base & 3) == 0) && ((P.baseB & 3) == 0) &&
            (((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B)) & 15u) == 0)) {
            const float4 *row = reinterpret_cast<const float4 *>(A + (unsigned)base);
            const float4 *wts = reinterpret_cast<const float4 *>(B + (unsigned)P.baseB);
            const unsigned K4 = K / 4;
            unsigned k = lane;
            for (; k + 96 < K4; k += 128) {
                const float4 a = __ldg(row + k), b = __ldg(row + k + 32), c = __ldg(row + k + 64), d = __ldg(row + k + 96);
                const float4 wa = __ldg(wts + k), wb = __ldg(wts + k + 32), wc = __ldg(wts + k + 64), wd = __ldg(wts + k + 96);
                s0 += (a.x * wa.x + a.y * wa.y) + (a.z * wa.z + a.w * wa.w); s1 += (b.x * wb.x + b.y * wb.y) + (b.z * wb.z + b.w * wb.w);
                s2 += (c.x * wc.x + c.y * wc.y) + (c.z * wc.z + c.w * wc.w); s3 += (d.x * wd.x + d.y * wd.y) + (d.z * wd.z + d.w * wd.w);
            }
            for (; k < K4; k += 32) { const float4 a = __ldg(row + k), wa = __ldg(wts + k); s0 += (a.x * wa.x + a.y * wa.y) + (a.z * wa.z + a.w * wa.w); }
            for (unsigned t = K4 * 4 + lane; t < K; t += 32) s1 = fmaf(__ldg(A + (unsigned)(base + (int)t)), __ldg(B + (unsigned)(P.baseB + (int)t)), s1);
        } else if (weighted) {
            unsigned k = lane;
            for (; k + 96 < K; k += 128) {
                s0 = fmaf(__ldg(A + (unsigned)(base + (int)k * ks)), __ldg(B + (unsigned)(P.baseB + (int)k * kb)), s0);
                s1 = fmaf(__ldg(A + (unsigned)(base + (int)(k + 32) * ks)), __ldg(B + (unsigned)(P.baseB + (int)(k + 32) * kb)), s1);
                s2 = fmaf(__ldg(A + (unsigned)(base + (int)(k + 64) * ks)), __ldg(B + (unsigned)(P.baseB + (int)(k + 64) * kb)), s2);
                s3 = fmaf(__ldg(A + (unsigned)(base + (int)(k + 96) * ks)), __ldg(B + (unsigned)(P.baseB + (int)(k + 96) * kb)), s3);
            }
            for (; k < K; k += 32) s0 = fmaf(__ldg(A + (unsigned)(base + (int)k * ks)), __ldg(B + (unsigned)(P.baseB + (int)k * kb)), s0);
        } else if (ks == 1 && ((base & 3) == 0) && ((reinterpret_cast<uintptr_t>(A) & 15u) == 0)) {
            const float4 *row = reinterpret_cast<const float4 *>(A + (unsigned)base);
            const unsigned K4 = K / 4;
            unsigned k = lane;
            for (; k + 96 < K4; k += 128) {
                const float4 a = __ldg(row + k), b = __ldg(row + k + 32), c = __ldg(row + k + 64), d = __ldg(row + k + 96);
                s0 += (a.x + a.y) + (a.z + a.w); s1 += (b.x + b.y) + (b.z + b.w);
                s2 += (c.x + c.y) + (c.z + c.w); s3 += (d.x + d.y) + (d.z + d.w);
            }
            for (; k < K4; k += 32) { const float4 a = __ldg(row + k); s0 += (a.x + a.y) + (a.z + a.w); }
            for (unsigned t = K4 * 4 + lane; t < K; t += 32) s1 += __ldg(A + (unsigned)(base + (int)t));
        } else {
            for (unsigned k = lane; k < K; k += 32) s0 += __ldg(A + (unsigned)(base + (int)k * ks));
        }
        float s = (s0 + s1) + (s2 + s3);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0) {
            const unsigned off = (unsigned)(P.baseO + p.o);
            float v = s * P.scale;
            if (P.accumulate) v += ptrs.out[off];
            ptrs.out[off] = v;
        }
    }
}

// Narrow contractions that stream a big operand: out[m, n] = sum_k A[m, k] B[n, k] with at most 36 columns n,
// one digit each for m, n and k, and B[k][n] rows of consecutive elements (the column blocks the optimisation
// pass lays out, or an argument read along its rows).  Every element of A is used by exactly one thread, so A
// goes from global memory straight into registers; only B is staged: 128 summation indices x 36 columns at a
// time in shared memory (16-byte asynchronous copies, two buffers), read with 128-bit loads.
//   A along k (A[m, k] consecutive in k): a warp owns two rows m, its lanes walk k four at a time (coalesced
//   128-bit loads), every lane keeps the sums of all columns for both rows and the warp adds them up at the end.
//   A along m (A[m, k] consecutive in m): a lane owns two rows m (32 apart) and walks all k of the block's slice;
//   the B values of a k are the same for the whole warp (broadcast loads).
// A summation split over blocks (grid.y) writes planes of partial sums like the tile kernel.
constexpr int SK_COLS = 36;        // columns held per row (9 groups of four)
constexpr int SK_KC = 128;         // summation indices per stage of B

__global__ void __launch_bounds__(256, 2)
tad_skinny_kernel(const __grid_constant__ TadcProgram P, const __grid_constant__ TadpPointers ptrs)
{
    __shared__ __align__(16) float bs[2][SK_KC * SK_COLS];
    const unsigned tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const float *__restrict__ A = ptrs.in[P.ptrA];
    const float *__restrict__ B = ptrs.in[P.ptrB];
    const unsigned Mext = (unsigned)P.M.extent, Next = (unsigned)P.N.extent, Kext = (unsigned)P.K.extent;
    const int sAm = P.M.n_digits ? P.M.sA[0] : 0, sAk = P.K.n_digits ? P.K.sA[0] : 0, sBk = P.K.n_digits ? P.K.sB[0] : 0;
    const unsigned ksplit = (unsigned)max(1, P.ksplit);
    const unsigned ks = blockIdx.y;
    const unsigned kbeg = ks * (unsigned)P.kchunk, kend = min(Kext, kbeg + (unsigned)P.kchunk);
    const int n_chunks = (int)((kend - kbeg + SK_KC - 1) / SK_KC);
    const bool along_k = P.modeA == TG_K;
    // rows of this thread
    unsigned m0, m1;
    if (along_k) { m0 = (blockIdx.x * 8u + warp) * 2u; m1 = m0 + 1u; }
    else { m0 = (blockIdx.x * 8u + warp) * 64u + lane; m1 = m0 + 32u; }
    const bool live0 = m0 < Mext, live1 = m1 < Mext;
    const unsigned a0 = (unsigned)(P.baseA + (int)(live0 ? m0 : 0u) * sAm), a1 = (unsigned)(P.baseA + (int)(live1 ? m1 : 0u) * sAm);
    float acc0[SK_COLS], acc1[SK_COLS];
#pragma unroll
    for (int n = 0; n < SK_COLS; ++n) { acc0[n] = 0.f; acc1[n] = 0.f; }
    // B chunk: rows of Next consecutive floats at B + baseB + k * sBk, copied as 16-byte pieces; columns beyond
    // Next and rows beyond the slice are zero
    const unsigned pieces = (Next + 3u) / 4u;                    // 16-byte pieces per row
    auto issue = [&](int chunk) {
        if (chunk < n_chunks) {
            float *dst = bs[chunk & 1];
            const unsigned k0 = kbeg + (unsigned)chunk * SK_KC;
            for (unsigned e = tid; e < SK_KC * (SK_COLS / 4); e += 256u) {
                const unsigned kl = e / (SK_COLS / 4), pc = e % (SK_COLS / 4);
                const bool ok = pc < pieces && k0 + kl < kend;
                // a row's last piece may reach past Next: the pass pads its rows to whole pieces, an argument read
                // along rows of a length that is no multiple of four does not take this kernel
                cp_async16(dst + kl * SK_COLS + pc * 4, B + (ok ? (unsigned)(P.baseB + (int)(k0 + kl) * sBk + (int)pc * 4) : 0u), ok);
            }
        }
        cp_async_commit();
    };
    // A along k: the values of the next chunk are loaded while the current one is multiplied
    float na[4] = {0.f, 0.f, 0.f, 0.f}, nb[4] = {0.f, 0.f, 0.f, 0.f};
    auto load_a = [&](int chunk) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const unsigned k = kbeg + (unsigned)chunk * SK_KC + lane + 32u * kk;
            const bool ok = chunk < n_chunks && k < kend;
            na[kk] = (ok && live0) ? __ldg(A + a0 + k) : 0.f;
            nb[kk] = (ok && live1) ? __ldg(A + a1 + k) : 0.f;
        }
    };
    issue(0);
    if (along_k) load_a(0);
    for (int ch = 0; ch < n_chunks; ++ch) {
        issue(ch + 1);
        float ga[4], gb[4];
        if (along_k) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) { ga[kk] = na[kk]; gb[kk] = nb[kk]; }
            load_a(ch + 1);
        }
        cp_async_wait<1>();
        __syncthreads();
        const float *bsc = bs[ch & 1];
        const unsigned k0 = kbeg + (unsigned)ch * SK_KC;
        if (along_k) {
            // lanes along k: lane l takes the summation indices l, l + 32, l + 64, l + 96 of the chunk for both rows
            // (coalesced loads of A; the rows of B a warp reads at a time are consecutive, 36 words apart: no bank
            // conflicts for its 128-bit loads)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const float *row = bsc + (lane + 32u * kk) * SK_COLS;
#pragma unroll
                for (int q = 0; q < SK_COLS / 4; ++q) {
                    const float4 b4 = *reinterpret_cast<const float4 *>(row + 4 * q);
                    acc0[4 * q] = fmaf(ga[kk], b4.x, acc0[4 * q]); acc0[4 * q + 1] = fmaf(ga[kk], b4.y, acc0[4 * q + 1]);
                    acc0[4 * q + 2] = fmaf(ga[kk], b4.z, acc0[4 * q + 2]); acc0[4 * q + 3] = fmaf(ga[kk], b4.w, acc0[4 * q + 3]);
                    acc1[4 * q] = fmaf(gb[kk], b4.x, acc1[4 * q]); acc1[4 * q + 1] = fmaf(gb[kk], b4.y, acc1[4 * q + 1]);
                    acc1[4 * q + 2] = fmaf(gb[kk], b4.z, acc1[4 * q + 2]); acc1[4 * q + 3] = fmaf(gb[kk], b4.w, acc1[4 * q + 3]);
                }
            }
        } else {
            // lanes along m: every k of the chunk, the loads of A eight indices ahead of their use
            const int kn = (int)min((unsigned)SK_KC, kend - k0);
            for (int kb = 0; kb < kn; kb += 8) {
                float ha[8], hb[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const bool ok = kb + u < kn;
                    const unsigned ko = (unsigned)((int)(k0 + kb + u) * sAk);
                    ha[u] = ok && live0 ? __ldg(A + a0 + ko) : 0.f;
                    hb[u] = ok && live1 ? __ldg(A + a1 + ko) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const float *row = bsc + (kb + u) * SK_COLS;      // rows past the slice are zero
#pragma unroll
                    for (int q = 0; q < SK_COLS / 4; ++q) {
                        const float4 b4 = *reinterpret_cast<const float4 *>(row + 4 * q);
                        acc0[4 * q] = fmaf(ha[u], b4.x, acc0[4 * q]); acc0[4 * q + 1] = fmaf(ha[u], b4.y, acc0[4 * q + 1]);
                        acc0[4 * q + 2] = fmaf(ha[u], b4.z, acc0[4 * q + 2]); acc0[4 * q + 3] = fmaf(ha[u], b4.w, acc0[4 * q + 3]);
                        acc1[4 * q] = fmaf(hb[u], b4.x, acc1[4 * q]); acc1[4 * q + 1] = fmaf(hb[u], b4.y, acc1[4 * q + 1]);
                        acc1[4 * q + 2] = fmaf(hb[u], b4.z, acc1[4 * q + 2]); acc1[4 * q + 3] = fmaf(hb[u], b4.w, acc1[4 * q + 3]);
                    }
                }
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();
    // ---- results ----
    const bool partial = ksplit > 1;
    float *__restrict__ out = partial ? ptrs.part : ptrs.out;
    const int sOm = P.M.n_digits ? P.M.sO[0] : 0, sOn = P.N.n_digits ? P.N.sO[0] : 0;
    auto store = [&](unsigned m, int n, float v) {
        if (partial) out[((size_t)ks * Mext + m) * Next + (unsigned)n] = v;
        else {
            const unsigned off = (unsigned)(P.baseO + (int)m * sOm + n * sOn);
            float r = epilogue(P, ptrs, v * P.scale, off);
            if (P.accumulate) r += out[off];
            out[off] = r;
        }
    };
    if (along_k) {
        // fixed-order butterfly over the lanes, then lane n stores column n
#pragma unroll
        for (int n = 0; n < SK_COLS; ++n) {
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                acc0[n] += __shfl_xor_sync(0xffffffffu, acc0[n], d);
                acc1[n] += __shfl_xor_sync(0xffffffffu, acc1[n], d);
            }
        }
#pragma unroll
        for (int n = 0; n < SK_COLS; ++n) {
            if ((unsigned)n < Next && (lane == (unsigned)(n & 31))) {
                if (live0) store(m0, n, acc0[n]);
                if (live1) store(m1, n, acc1[n]);
            }
        }
    } else {
#pragma unroll
        for (int n = 0; n < SK_COLS; ++n) {
            if ((unsigned)n < Next) {
                if (live0) store(m0, n, acc0[n]);
                if (live1) store(m1, n, acc1[n]);
            }
        }
    }
}

// Plain or weighted sums of an operand that is consecutive along its row index:
//     out[m] = sum_k A[m + k * stride] (* B[k]),   a thread per m, a slice of k per block row (grid.y);
// consecutive threads read consecutive elements, four loads in flight per thread.  Slices write planes of
// partial sums that tad_contract_reduce adds in order.
__global__ void __launch_bounds__(256)
tad_colsum_kernel(const __grid_constant__ TadcProgram P, const __grid_constant__ TadpPointers ptrs)
{
    const unsigned m = blockIdx.x * 256u + threadIdx.x;
    const unsigned Mext = (unsigned)P.M.extent, K = (unsigned)P.K.extent;
    if (m >= Mext) return;
    const float *__restrict__ A = ptrs.in[P.ptrA];
    const bool weighted = P.ptrB >= 0;
    const float *__restrict__ B = weighted ? ptrs.in[P.ptrB] : A;
    const int ks = P.K.sA[0], kb = P.K.sB[0];
    const unsigned kbeg = blockIdx.y * (unsigned)P.kchunk, kend = min(K, kbeg + (unsigned)P.kchunk);
    const int base = P.baseA + (int)m * P.M.sA[0];
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    unsigned k = kbeg;
    for (; k + 7 < kend; k += 8) {
        float a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) a[u] = __ldg(A + (unsigned)(base + (int)(k + u) * ks));
        if (weighted) {
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] *= __ldg(B + (unsigned)(P.baseB + (int)(k + u) * kb));
        }
        s0 += a[0] + a[4]; s1 += a[1] + a[5]; s2 += a[2] + a[6]; s3 += a[3] + a[7];
    }
    for (; k < kend; ++k) {
        const float a0 = __ldg(A + (unsigned)(base + (int)k * ks));
        s0 = weighted ? fmaf(a0, __ldg(B + (unsigned)(P.baseB + (int)k * kb)), s0) : s0 + a0;
    }
    const float s = (s0 + s1) + (s2 + s3);
    if (P.ksplit > 1) ptrs.part[(size_t)blockIdx.y * Mext + m] = s;
    else {
        const unsigned off = (unsigned)(P.baseO + (int)m * P.M.sO[0]);
        float v = s * P.scale;
        if (P.accumulate) v += ptrs.out[off];
        ptrs.out[off] = v;
    }
}

template <int BM, int BN, int TM, int TN>
cudaError_t launch_shape(const TadcProgram &P, const TadpPointers &ptrs, cudaStream_t stream)
{
    using C = Cfg<BM, BN, TM, TN>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    auto kern = tad_contract_kernel<BM, BN, TM, TN>;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    const unsigned tiles_m = ((unsigned)P.M.extent + BM - 1) / BM, tiles_n = ((unsigned)P.N.extent + BN - 1) / BN;
    dim3 grid(tiles_m * tiles_n, (unsigned)std::max(1, P.ksplit), (unsigned)P.Z.extent);
    kern<<<grid, C::NT, C::SMEM, stream>>>(P, ptrs, tiles_m, tiles_n);
    return cudaGetLastError();
}

}  // namespace

cudaError_t tad_launch_contract(const TadcProgram &P, const TadpPointers &ptrs, unsigned sms, cudaStream_t stream)
{
    if (P.M.extent <= 0 || P.N.extent <= 0 || P.Z.extent <= 0) return cudaSuccess;
    if (P.shape == 5) {
        const unsigned rows_per_block = P.modeA == TG_K ? 16u : 512u;
        dim3 grid(((unsigned)P.M.extent + rows_per_block - 1u) / rows_per_block, (unsigned)std::max(1, P.ksplit), 1u);
        tad_skinny_kernel<<<grid, 256, 0, stream>>>(P, ptrs);
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess && P.ksplit > 1) {
            const unsigned long long cells = (unsigned long long)P.M.extent * P.N.extent;
            const unsigned blocks = (unsigned)std::min<unsigned long long>((cells + 255) / 256, (unsigned long long)sms * 8);
            tad_contract_reduce<<<blocks, 256, 0, stream>>>(P, ptrs);
            e = cudaGetLastError();
        }
        return e;
    }
    if (P.shape == 6) {
        dim3 grid(((unsigned)P.M.extent + 255u) / 256u, (unsigned)std::max(1, P.ksplit), 1u);
        tad_colsum_kernel<<<grid, 256, 0, stream>>>(P, ptrs);
        cudaError_t e = cudaGetLastError();
        if (e == cudaSuccess && P.ksplit > 1) {
            const unsigned blocks = (unsigned)std::min<unsigned long long>(((unsigned long long)P.M.extent + 255) / 256, (unsigned long long)sms * 8);
            tad_contract_reduce<<<blocks, 256, 0, stream>>>(P, ptrs);
            e = cudaGetLastError();
        }
        return e;
    }
    if (P.shape == 4) {
        const unsigned warps = (unsigned)P.M.extent;
        const unsigned blocks = std::min((warps + 7u) / 8u, sms * 16u);
        tad_rowsum_kernel<<<blocks, 256, 0, stream>>>(P, ptrs);
        return cudaGetLastError();
    }
    cudaError_t e = P.shape == 1 ? launch_shape<128, 32, 8, 4>(P, ptrs, stream)
                  : P.shape == 3 ? launch_shape<128, 36, 8, 4>(P, ptrs, stream)
                  : P.shape == 2 ? launch_shape<128, 64, 8, 4>(P, ptrs, stream) : launch_shape<128, 128, 8, 8>(P, ptrs, stream);
    if (e != cudaSuccess) return e;
    if (P.ksplit > 1) {
        const unsigned long long cells = (unsigned long long)P.M.extent * P.N.extent * P.Z.extent;
        const unsigned blocks = (unsigned)std::min<unsigned long long>((cells + 255) / 256, (unsigned long long)sms * 8);
        tad_contract_reduce<<<blocks, 256, 0, stream>>>(P, ptrs);
        e = cudaGetLastError();
    }
    return e;
}

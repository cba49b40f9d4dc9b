// Contraction planner (host only): recognises a kernel whose term is a product of two index
// expressions under summations and rewrites it as one or several contraction programs
// (contract.h) for the tile kernel.
//
// The loop variables of the kernel are split by which of the two factors reads them: variables
// that only the first factor reads index the rows m of the tile, variables that only the second
// reads (or neither) index its columns n, variables both read and that are not summed form a batch
// index, and the summed variables form k.  Every index expression is affine (Sec. 5.1), so each
// factor's element offset is a sum of one part per group, which is all the tile kernel needs.
//
// A summation loop whose bounds move with another variable v as a band,
//     (c_lo + a v) / d  <=  z  <=  (c_hi + a v) / d,
// (the taps of a transposed strided convolution: Sec. 5.1's range form with a rational slope) is
// brought to fixed bounds by the substitution  v = d' v' + p,  z = a' v' + r  with a / d = a' / d'
// in lowest terms: for every residue p the offset r runs over a fixed range, so each residue
// class becomes a contraction of its own; the remaining constant bounds of z turn into a guard
// that reads operand elements outside them as zero.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <numeric>

#include "gen.h"

namespace tad {

namespace {

int32_t fit(int64_t v) { if (std::llabs(v) >= (int64_t(1) << 31)) throw Overflow(); return (int32_t)v; }

struct Digit { int var; int64_t ext, sA, sB, sO; };

bool fill_group(TadcGroup &G, std::vector<Digit> &ds, const AGuard *ga, const AGuard *gb)
{
    if ((int)ds.size() > TADC_MAX_DIGITS) return false;
    G = TadcGroup{};
    G.n_digits = (int32_t)ds.size();
    int64_t extent = 1;
    for (size_t d = 0; d < ds.size(); ++d) {
        G.ext[d] = fit(ds[d].ext);
        G.sA[d] = fit(ds[d].sA); G.sB[d] = fit(ds[d].sB); G.sO[d] = fit(ds[d].sO);
        G.gA[d] = ga ? fit(ga->coef[ds[d].var]) : 0;
        G.gB[d] = gb ? fit(gb->coef[ds[d].var]) : 0;
        extent = mul_ck(extent, ds[d].ext);
    }
    G.extent = fit(extent);
    return true;
}

}  // namespace

// builds one contraction program from a system whose loops all have fixed ranges
bool emit_program(const System &s0, float scale, int accumulate, bool allow_split, bool strict_fill, TadcProgram &P, std::string &text)
{
    System s = s0;
    const int nv = (int)s.vars.size();
    if (s.A.ptr < 0) std::swap(s.A, s.B);                  // an operand of ones plays B
    // which factor plays A: the variable along which the output is contiguous should index columns
    int contiguous = -1;
    for (int v = 0; v < nv; ++v)
        if (!s.vars[v].reduce && s.O.coef[v] != 0 && s.vars[v].ext > 1 &&
            (contiguous < 0 || std::llabs(s.O.coef[v]) < std::llabs(s.O.coef[contiguous]))) contiguous = v;
    bool b_has_rows = false;                               // B reads some variable that is not summed
    for (int v = 0; v < nv; ++v) if (!s.vars[v].reduce && s.vars[v].ext > 1 && s.B.coef[v] != 0) b_has_rows = true;
    if (contiguous >= 0 && s.A.coef[contiguous] != 0 && s.B.coef[contiguous] == 0 && s.B.ptr >= 0 && b_has_rows) std::swap(s.A, s.B);
    std::vector<Digit> dm, dn, dk, dz;
    for (int v = 0; v < nv; ++v) {
        if (s.vars[v].ext == 1) continue;                  // a single value: nothing to index
        Digit d{v, s.vars[v].ext, s.A.coef[v], s.B.coef[v], s.O.coef[v]};
        if (s.vars[v].reduce) dk.push_back(d);
        else if (d.sA != 0 && d.sB != 0) dz.push_back(d);
        else if (d.sA != 0) dm.push_back(d);
        else dn.push_back(d);
    }
    auto mag = [](int64_t a) { return a == 0 ? INT64_MAX : std::llabs(a); };
    // fastest digit last: rows by their stride in the operand, columns by their stride in the output
    std::stable_sort(dm.begin(), dm.end(), [&](const Digit &x, const Digit &y) { return mag(x.sA) > mag(y.sA); });
    std::stable_sort(dn.begin(), dn.end(), [&](const Digit &x, const Digit &y) {
        return mag(x.sO) != mag(y.sO) ? mag(x.sO) > mag(y.sO) : mag(x.sB) > mag(y.sB); });
    std::stable_sort(dk.begin(), dk.end(), [&](const Digit &x, const Digit &y) {
        return std::min(mag(x.sA), mag(x.sB)) > std::min(mag(y.sA), mag(y.sB)); });
    // guards: at most one per operand; a guard belongs to an operand whose groups hold all its variables
    const AGuard *ga = nullptr, *gb = nullptr;
    auto in_group = [&](const std::vector<Digit> &g, int v) { for (const Digit &d : g) if (d.var == v) return true; return false; };
    for (const AGuard &gd : s.guards) {
        bool fits_a = true, fits_b = true;
        for (int v = 0; v < nv; ++v) {
            if (!gd.coef[v] || s.vars[v].ext == 1) continue;
            if (in_group(dn, v)) fits_a = false;
            if (in_group(dm, v)) fits_b = false;
        }
        if (fits_b && !gb) gb = &gd;
        else if (fits_a && !ga) ga = &gd;
        else return false;
    }
    // every offset the kernel can form must lie inside its tensor: interval check over the digit ranges
    // (an operand under a guard is checked over the guarded range of its guard expression only when the
    // guard is the identity on one digit pair, so it is skipped here: the guard itself bounds the reads)
    auto in_range = [&](const AMap &m, bool guarded) {
        if (guarded || m.ptr < 0) return true;
        int64_t lo = m.base, hi = m.base;
        for (int v = 0; v < nv; ++v) {
            if (s.vars[v].ext <= 1) { if (s.vars[v].ext <= 0) return true; continue; }
            const int64_t span = mul_ck(m.coef[v], s.vars[v].ext - 1);
            if (span < 0) lo = add_ck(lo, span); else hi = add_ck(hi, span);
        }
        return lo >= 0 && hi < m.limit;
    };
    if (!in_range(s.A, ga != nullptr) || !in_range(s.B, gb != nullptr) || !in_range(s.O, false)) {
        // a masked index expression iterates a bounding box of its image lattice and the interpreter skips the
        // elements without terms; the tile kernel would touch them, so such a kernel stays with the interpreter
        if (s.loose_box) return false;
        std::string what = "internal: contraction offsets leave their tensor:";
        for (const AMap *m : {&s.A, &s.B, &s.O}) {
            what += " [ptr " + std::to_string(m->ptr) + " base " + std::to_string(m->base) + " limit " + std::to_string(m->limit) + " coef";
            for (int v = 0; v < nv; ++v) if (m->coef[v]) what += " " + std::to_string(v) + ":" + std::to_string(m->coef[v]) + "x" + std::to_string(s.vars[v].ext);
            what += "]";
        }
        throw BadExpr(what);
    }
    P = TadcProgram{};
    if (!fill_group(P.M, dm, ga, nullptr) || !fill_group(P.N, dn, nullptr, gb) || !fill_group(P.K, dk, ga, gb) ||
        !fill_group(P.Z, dz, ga, gb)) return false;
    if (P.Z.extent > 65535) return false;
    P.ptrA = s.A.ptr; P.ptrB = s.B.ptr;
    P.baseA = fit(s.A.base); P.baseB = fit(s.B.base); P.baseO = fit(s.O.base);
    P.guardA = ga ? 1 : 0; P.guardA_c0 = ga ? fit(ga->c0) : 0; P.guardA_ext = ga ? fit(ga->ext) : 1;
    P.guardB = gb ? 1 : 0; P.guardB_c0 = gb ? fit(gb->c0) : 0; P.guardB_ext = gb ? fit(gb->ext) : 1;
    P.scale = scale; P.accumulate = accumulate;
    // tile shape: narrow column tiles for narrow outputs
    P.shape = P.N.extent <= 32 ? 1 : P.N.extent <= 36 ? 3 : P.N.extent <= 64 ? 2 : 0;
    const int64_t BM = 128, BN = P.shape == 1 ? 32 : P.shape == 3 ? 36 : P.shape == 2 ? 64 : 128;
    const int64_t tiles_m = (P.M.extent + BM - 1) / BM, tiles_n = (P.N.extent + BN - 1) / BN;
    const double fill = (double)P.M.extent * P.N.extent / ((double)tiles_m * BM * tiles_n * BN);
    // one output column: plain or weighted sums of A (B is ones or a vector over k), run at memory speed by a warp
    // per row (A along k) or a thread per row (A along m)
    const bool one_column = P.N.extent == 1 && P.Z.extent == 1 && P.K.n_digits <= 1 && !P.guardA && !P.guardB && P.M.extent >= 1024;
    const bool col_sums = one_column && P.M.n_digits == 1 && P.M.sA[0] == 1 && P.K.n_digits == 1 && std::llabs((int64_t)P.K.sA[0]) != 1;
    const bool row_sums = one_column && !col_sums;
    if (!one_column && fill < (strict_fill ? 0.15 : 0.05)) return false;    // mostly empty tiles: the interpreter's schedules do better
    // gather modes: the one whose warp-wide copy touches fewer 128-byte lines (lanes along the row index:
    // 32 rows at one summation index; lanes along the summation index: 2 rows x 16 indices)
    auto mode_of = [&](const std::vector<Digit> &rows, bool second, const AGuard *gd, int64_t base) {
        auto st = [&](const Digit &d) { return std::llabs(second ? d.sB : d.sA); };
        // longest run of consecutive elements along the fastest digits of a group
        auto run_of = [&](const std::vector<Digit> &ds) {
            int64_t run = 1;
            for (int d = (int)ds.size() - 1; d >= 0; --d) {
                if (st(ds[d]) != run) break;
                run *= ds[d].ext;
            }
            return run;
        };
        const int64_t rs = rows.empty() ? 0 : st(rows.back());
        const int64_t ks = dk.empty() ? 0 : st(dk.back());
        auto lines = [&](int64_t stride, int64_t run, int64_t ext, int64_t n) {     // n consecutive indices of a group
            if (stride == 0) return int64_t(1);
            if (stride == 1) return run >= n ? int64_t(1) : (n + run - 1) / run;
            if (ext >= n) return std::min<int64_t>(n, (n * stride + 31) / 32);
            return (n + ext - 1) / ext * std::max<int64_t>(1, (ext * stride + 31) / 32);
        };
        const int64_t lines_row = lines(rs, run_of(rows), rows.empty() ? 1 : rows.back().ext, 32);
        const int64_t lines_k = lines(ks, run_of(dk), dk.empty() ? 1 : dk.back().ext, 16) * (rs * 2 <= 32 ? 1 : 2);
        if (lines_k < lines_row) return TG_K;
        if (rs == 1) {
            bool wide = (second ? rows.back().sB : rows.back().sA) == 1 && rows.back().ext % 4 == 0 && base % 4 == 0 &&
                        !(gd && gd->coef[rows.back().var]);
            for (size_t d = 0; d + 1 < rows.size(); ++d) if (st(rows[d]) % 4) wide = false;
            for (const Digit &d : dk) if (st(d) % 4) wide = false;
            for (const Digit &d : dz) if (st(d) % 4) wide = false;
            if (wide) return TG_ROW16;
        }
        return TG_ROW;
    };
    P.modeA = mode_of(dm, false, ga, s.A.base);
    P.modeB = s.B.ptr < 0 ? TG_ROW : mode_of(dn, true, gb, s.B.base);
    // output: four consecutive columns are four consecutive aligned elements
    P.out_vec4 = 0;
    if (!dn.empty() && dn.back().sO == 1 && dn.back().ext % 4 == 0 && s.O.base % 4 == 0) {
        P.out_vec4 = 1;
        for (size_t d = 0; d + 1 < dn.size(); ++d) if (dn[d].sO % 4) P.out_vec4 = 0;
        for (const Digit &d : dm) if (d.sO % 4) P.out_vec4 = 0;
        for (const Digit &d : dz) if (d.sO % 4) P.out_vec4 = 0;
    }
    // summation split: enough blocks for two per SM when the tiles alone are too few
    const int64_t blocks = tiles_m * tiles_n * P.Z.extent;
    const int64_t kstages = (P.K.extent + TADC_BK - 1) / TADC_BK;
    int64_t split = 1;
    if (allow_split && blocks < 222 && kstages >= 16) {
        // the number of chunks that fills whole waves of resident blocks best (two blocks per SM), every
        // chunk at least eight stages long; fewer chunks win ties (less partial-sum traffic)
        const int64_t wave = P.shape == 0 ? 296 : P.shape == 2 ? 444 : 592;
        const int64_t cells = (int64_t)P.M.extent * P.N.extent * P.Z.extent;
        double best = 0;
        for (int64_t s = 1; s <= std::min<int64_t>(kstages / 8, 256); ++s) {
            if (s > 1 && s * cells > (int64_t(1) << 25)) break;                     // <= 128 MB of partial sums
            const int64_t grid = blocks * s;
            const double eff = (double)grid / (double)((grid + wave - 1) / wave * wave);
            if (eff > best + 0.02) { best = eff; split = s; }
        }
    }
    if (row_sums) { P.shape = 4; split = 1; }
    if (col_sums) {
        // a thread per row, blocks of 256 rows: the summation is split to fill the GPU
        P.shape = 6;
        const int64_t row_blocks = (P.M.extent + 255) / 256;
        split = allow_split ? std::max<int64_t>(1, std::min<int64_t>((592 + row_blocks - 1) / row_blocks, P.K.extent / 64)) : 1;
        const int64_t cells = (int64_t)P.M.extent;
        while (split > 1 && split * cells > (int64_t(1) << 25)) --split;
        const int64_t per = (P.K.extent + split - 1) / split;
        P.kchunk = fit(std::max<int64_t>(per, 1));
        P.ksplit = fit((P.K.extent + P.kchunk - 1) / P.kchunk);
    }
    // the streaming kernel for narrow contractions (see tad_skinny_kernel): one digit per group, B rows of consecutive,
    // 16-byte aligned elements, A consecutive along k (128-bit loads) or along m
    if (!one_column && s.B.ptr >= 0 && !ga && !gb && P.Z.extent == 1 && P.N.extent >= 2 && P.N.extent <= 36 && P.M.n_digits == 1 &&
        P.K.n_digits == 1 && P.N.n_digits == 1 && P.N.sB[0] == 1 && P.M.extent >= 512 && P.K.extent >= 512) {
        const int64_t sBk = P.K.sB[0], sAk = P.K.sA[0], sAm = P.M.sA[0];
        const bool b_ok = sBk > 0 && sBk % 4 == 0 && s.B.base % 4 == 0 && (P.N.extent % 4 == 0 || sBk >= (P.N.extent + 3) / 4 * 4);
        // (A along k is left to the tiles: with the lanes along k every lane reads its own rows of B from shared
        // memory, which that memory cannot deliver at the rate of the multiply-adds; the kernel keeps the path)
        const bool along_k = false && sAk == 1;
        const bool along_m = sAm == 1;
        if (b_ok && (along_k || along_m)) {
            P.shape = 5;
            P.modeA = along_k ? TG_K : TG_ROW;
            const int64_t row_blocks = along_k ? (P.M.extent + 15) / 16 : (P.M.extent + 511) / 512;
            split = 1;
            if (allow_split && row_blocks < 222) split = std::max<int64_t>(1, std::min<int64_t>(296 / row_blocks, P.K.extent / 512));
            const int64_t cells = (int64_t)P.M.extent * P.N.extent;
            while (split > 1 && split * cells > (int64_t(1) << 25)) --split;
            const int64_t per128 = ((P.K.extent + split - 1) / split + 127) / 128 * 128;
            P.kchunk = fit(per128);
            P.ksplit = fit((P.K.extent + per128 - 1) / per128);
        }
    }
    if (P.shape != 5 && P.shape != 6) {
    split = std::max<int64_t>(1, split);
    const int64_t per = ((kstages + split - 1) / split) * TADC_BK;
    P.kchunk = fit(std::max<int64_t>(per, TADC_BK));
    P.ksplit = fit(std::max<int64_t>(1, (P.K.extent + P.kchunk - 1) / P.kchunk));
    if (P.ksplit <= 1) { P.ksplit = 1; P.kchunk = fit(std::max<int64_t>(kstages, 1) * TADC_BK); }
    }
    if (P.shape == 5 && P.ksplit <= 1) { P.ksplit = 1; P.kchunk = fit((P.K.extent + 127) / 128 * 128); }
    char line[320];
    auto group_text = [&](const char *name, const TadcGroup &G) {
        std::string t = std::string("  ") + name + ":";
        for (int d = 0; d < G.n_digits; ++d) {
            std::snprintf(line, sizeof line, " [ext %d sA %d sB %d sO %d]", G.ext[d], G.sA[d], G.sB[d], G.sO[d]);
            t += line;
        }
        return t + "\n";
    };
    std::snprintf(line, sizeof line, "; contraction %d x %d x %d (batch %d): A=ptr %d mode %d guard %d, B=ptr %d mode %d guard %d, tile %s, ksplit %d x %d, vec4 %d, scale %g, accumulate %d\n",
                  P.M.extent, P.N.extent, P.K.extent, P.Z.extent, P.ptrA, P.modeA, P.guardA, P.ptrB, P.modeB, P.guardB,
                  P.shape == 6 ? "column sums" : P.shape == 5 ? "streamed" : P.shape == 4 ? "row sums" : P.shape == 1 ? "128x32" : P.shape == 3 ? "128x36" : P.shape == 2 ? "128x64" : "128x128", P.ksplit, P.kchunk, P.out_vec4, (double)P.scale, P.accumulate);
    text += line;
    text += group_text("m", P.M) + group_text("n", P.N) + group_text("k", P.K) + group_text("z", P.Z);
    return true;
}

bool try_contraction(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
                     const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards)
{
    if (g.p.opt.debug_bounds || !guards.empty() || root < 0) return false;
    const TadpProgram &prog = k.prog;
    float cfac = 1.f;
    if (scale >= 0) { if (g.inst[scale].op != I_CONST) return false; cfac = g.inst[scale].imm; }
    const int nv = (int)g.vars.size();
    // ---- the term: constant factors, sums, then a product of two loads ----
    std::vector<int64_t> vlo(nv, 0), vext(nv, 1);
    std::vector<bool> reduce(nv, false), seen(nv, false);
    for (int v = 0; v < g.n_outer; ++v) { vlo[v] = prog.outer_lo[v]; vext[v] = prog.outer_ext[v]; seen[v] = true; }
    int cur = root;
    for (;;) {
        const Inst &in = g.inst[cur];
        if (in.op == I_SUM) { vlo[in.var] = in.lo; vext[in.var] = std::max<int64_t>(0, in.hi - in.lo + 1); reduce[in.var] = true; seen[in.var] = true; cur = in.a; }
        else if (in.op == I_MULC) { cfac *= in.imm; cur = in.a; }
        else if (in.op == I_NEG) { cfac = -cfac; cur = in.a; }
        else break;
    }
    auto as_load = [&](int i) {
        for (;;) {
            const Inst &in = g.inst[i];
            if (in.op == I_MULC) { cfac *= in.imm; i = in.a; }
            else if (in.op == I_NEG) { cfac = -cfac; i = in.a; }
            else return in.op == I_LOAD ? in.load : -1;
        }
    };
    int la = -1, lb = -1;
    if (g.inst[cur].op == I_MUL) { la = as_load(g.inst[cur].a); lb = as_load(g.inst[cur].b); }
    else if (g.inst[cur].op == I_SQR) {
        // (c L)^2 = c^2 L L
        const float outer_c = cfac;
        cfac = 1.f;
        la = lb = as_load(g.inst[cur].a);
        cfac = outer_c * cfac * cfac;
    }
    if (la < 0 || lb < 0) return false;
    // ---- kernel-coordinate loops: fixed ranges, or one band ----
    struct Band { int z, v; int64_t a, d, c_lo, c_hi; int64_t zmin, zmax; bool has_min, has_max; };
    bool have_band = false; Band band{};
    for (int l = 0; l < g.kappa; ++l) {
        const int z = g.n_outer + g.zorder[l];
        reduce[z] = true; seen[z] = true;
        auto constant = [&](const TadpRow &r) { for (int v = 0; v < TADP_MAX_VARS; ++v) if (r.coef[v]) return false; return true; };
        bool all_const = true;
        for (const TadpRow &r : lower[l]) all_const = all_const && constant(r);
        for (const TadpRow &r : upper[l]) all_const = all_const && constant(r);
        if (lower[l].empty() || upper[l].empty()) return false;
        if (all_const) {
            int64_t lo = INT64_MIN, hi = INT64_MAX;
            for (const TadpRow &r : lower[l]) lo = std::max(lo, ceil_div(r.c0, r.den));
            for (const TadpRow &r : upper[l]) hi = std::min(hi, floor_div(r.c0, r.den));
            vlo[z] = lo; vext[z] = std::max<int64_t>(0, hi - lo + 1);
            continue;
        }
        if (have_band) return false;
        // one lower and one upper row with the same slope on one variable; every other row constant
        const TadpRow *rl = nullptr, *rh = nullptr;
        int64_t zmin = 0, zmax = 0; bool has_min = false, has_max = false;
        for (const TadpRow &r : lower[l]) {
            if (constant(r)) { const int64_t c = ceil_div(r.c0, r.den); zmin = has_min ? std::max(zmin, c) : c; has_min = true; }
            else if (!rl) rl = &r; else return false;
        }
        for (const TadpRow &r : upper[l]) {
            if (constant(r)) { const int64_t c = floor_div(r.c0, r.den); zmax = has_max ? std::min(zmax, c) : c; has_max = true; }
            else if (!rh) rh = &r; else return false;
        }
        if (!rl || !rh) return false;
        int bv = -1;
        for (int v = 0; v < TADP_MAX_VARS; ++v) {
            if (!rl->coef[v] && !rh->coef[v]) continue;
            if (bv >= 0) return false;
            bv = v;
        }
        // same slope: a_l / d_l == a_h / d_h; bring both rows to the common denominator
        const int64_t dl = rl->den, dh = rh->den, al = rl->coef[bv], ah = rh->coef[bv];
        if (al * dh != ah * dl) return false;
        const int64_t d = dl / gcd64(dl, dh) * dh;
        band = Band{z, bv, al * (d / dl), d, rl->c0 * (d / dl), rh->c0 * (d / dh), zmin, zmax, has_min, has_max};
        if ((band.c_hi - band.c_lo) / band.d > 64) return false;     // not a narrow band
        have_band = true;
    }
    for (int v = 0; v < nv; ++v) if (!seen[v]) return false;
    const TadpLoad &LA = g.loads[la], &LB = g.loads[lb];
    // ---- the affine system, every variable counted from zero ----
    System base;
    base.vars.resize(nv);
    base.A.ptr = LA.ptr; base.B.ptr = LB.ptr;
    base.A.base = LA.base; base.B.base = LB.base; base.O.base = prog.out_base;
    base.loose_box = prog.write_only_live != 0;
    base.A.limit = LA.limit; base.B.limit = LB.limit; base.O.limit = prog.out_limit;
    base.A.coef.assign(nv, 0); base.B.coef.assign(nv, 0); base.O.coef.assign(nv, 0);
    for (int v = 0; v < nv; ++v) {
        base.vars[v] = AVar{vext[v], reduce[v]};
        base.A.coef[v] = LA.coef[v]; base.B.coef[v] = LB.coef[v];
        base.O.coef[v] = v < g.n_outer ? prog.out_coef[v] : 0;
    }
    auto shift = [&](System &s, int v, int64_t by) {      // variable v := by + v
        s.A.base = add_ck(s.A.base, mul_ck(s.A.coef[v], by));
        s.B.base = add_ck(s.B.base, mul_ck(s.B.coef[v], by));
        s.O.base = add_ck(s.O.base, mul_ck(s.O.coef[v], by));
        for (AGuard &gd : s.guards) gd.c0 = add_ck(gd.c0, mul_ck(gd.coef[v], by));
    };
    std::vector<System> systems;
    if (!have_band) {
        for (int v = 0; v < nv; ++v) shift(base, v, vlo[v]);
        systems.push_back(base);
    } else {
        // v = vlo + w with w = d' w' + p; the band in terms of w: (c + a vlo + a w) / d
        const int v = band.v, z = band.z;
        if (v == z) return false;
        for (int u = 0; u < nv; ++u) if (u != z) shift(base, u, vlo[u]);
        const int64_t c_lo = add_ck(band.c_lo, mul_ck(band.a, vlo[v])), c_hi = add_ck(band.c_hi, mul_ck(band.a, vlo[v]));
        const int64_t gq = gcd64(std::llabs(band.a), band.d);
        const int64_t a1 = band.a / gq, d1 = band.d / gq;
        if (d1 > 8) return false;
        for (int64_t p = 0; p < d1; ++p) {
            System s = base;
            const int64_t r_lo = ceil_div(add_ck(c_lo, mul_ck(band.a, p)), band.d);
            const int64_t r_hi = floor_div(add_ck(c_hi, mul_ck(band.a, p)), band.d);
            const int64_t wext = vext[v] > p ? (vext[v] - p + d1 - 1) / d1 : 0;
            // substitute  w = d1 w' + p,  z = a1 w' + r_lo + r
            auto subst = [&](AMap &m) {
                m.base = add_ck(m.base, add_ck(mul_ck(m.coef[v], p), mul_ck(m.coef[z], r_lo)));
                m.coef[v] = add_ck(mul_ck(m.coef[v], d1), mul_ck(m.coef[z], a1));
            };
            subst(s.A); subst(s.B); subst(s.O);
            s.vars[v].ext = wext;
            s.vars[z].ext = std::max<int64_t>(0, r_hi - r_lo + 1);
            if (band.has_min || band.has_max) {
                // zmin <= z <= zmax with z = a1 w' + r_lo + r
                if (!band.has_min || !band.has_max) return false;
                AGuard gd;
                gd.coef.assign(nv, 0);
                gd.coef[v] = a1; gd.coef[z] = 1;
                gd.c0 = r_lo - band.zmin;
                gd.ext = band.zmax - band.zmin + 1;
                if (gd.ext <= 0) s.vars[z].ext = 0;
                gd.ext = std::max<int64_t>(gd.ext, 1);
                s.guards.push_back(gd);
            }
            systems.push_back(s);
        }
    }
    std::vector<TadcProgram> progs;
    std::string text;
    for (const System &s : systems) {
        bool empty_out = false;
        for (int v = 0; v < nv; ++v) if (!s.vars[v].reduce && s.vars[v].ext <= 0) empty_out = true;
        if (empty_out) continue;
        TadcProgram P;
        if (!emit_program(s, cfac, prog.accumulate, allow_split, true, P, text)) return false;
        progs.push_back(P);
    }
    if (progs.empty()) return false;
    k.contract = progs;
    k.listing = text;
    k.vec = 0; k.vec_u = 0;
    return true;
}

}  // namespace tad

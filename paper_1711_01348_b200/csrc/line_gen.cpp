// Recogniser for line-sum programs (line.h): a gradient kernel (one or two summation loops with the bound rows
// of Sec. 4.2) whose term is a product of index expressions and constants, with a factor outside the sums that
// is again such a product.  After the function tables of the optimisation pass most derivative terms have this
// form (df times pre-evaluated functions of the arguments), and the kernel runs them without interpretation.
#include <algorithm>
#include <cstring>
#include <functional>

#include "gen.h"
#define LFAIL return false

namespace tad {

bool try_line(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
              const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards)
{
    if (g.p.opt.debug_bounds || root < 0 || g.kappa < 1 || g.kappa > 2 || g.n_outer < 1 || g.n_outer > 4) return false;
    TadpProgram &prog = k.prog;
    // ---- the term and the outer factor: products of loads and constants ----
    float cterm = 1.f, cscale = 1.f;
    std::vector<int> loads, sloads;
    std::function<bool(int, float &, std::vector<int> &, size_t)> flat = [&](int i, float &c, std::vector<int> &out, size_t cap) {
        const Inst in = g.inst[i];
        switch (in.op) {
        case I_MUL: return flat(in.a, c, out, cap) && flat(in.b, c, out, cap);
        case I_MULC: c *= in.imm; return flat(in.a, c, out, cap);
        case I_NEG: c = -c; return flat(in.a, c, out, cap);
        case I_SQR: return flat(in.a, c, out, cap) && flat(in.a, c, out, cap);
        case I_CONST: c *= in.imm; return true;
        case I_LOAD: out.push_back(in.load); return out.size() <= cap;
        default: return false;
        }
    };
    if (!flat(root, cterm, loads, TADL_MAX_LOADS) || loads.empty()) LFAIL;
    if (scale >= 0 && !flat(scale, cscale, sloads, 2)) LFAIL;
    const int z_id[2] = {g.n_outer + g.zorder[0], g.kappa == 2 ? g.n_outer + g.zorder[1] : -1};
    auto conv_load = [&](const TadpLoad &L, TadlLoad &out) {
        out = TadlLoad{};
        out.ptr = L.ptr; out.base = L.base;
        for (int v = 0; v < TADP_MAX_VARS; ++v) {
            if (!L.coef[v]) continue;
            if (v < g.n_outer) out.coef[v] = L.coef[v];
            else if (v == z_id[0]) out.cz[0] = L.coef[v];
            else if (v == z_id[1]) out.cz[1] = L.coef[v];
            else return false;
        }
        return true;
    };
    auto conv_row = [&](const TadpRow &R, int loop, TadlRow &out) {
        out = TadlRow{};
        out.den = R.den; out.c0 = R.c0;
        for (int v = 0; v < TADP_MAX_VARS; ++v) {
            if (!R.coef[v]) continue;
            if (v < g.n_outer) out.coef[v] = R.coef[v];
            else if (loop == 1 && v == z_id[0]) out.cz = R.coef[v];
            else return false;
        }
        return true;
    };
    TadlProgram P{};
    P.n_outer = g.n_outer; P.n_loops = g.kappa;
    for (int l = 0; l < g.kappa; ++l) {
        if (lower[l].empty() || upper[l].empty() || lower[l].size() > TADL_MAX_ROWS || upper[l].size() > TADL_MAX_ROWS) LFAIL;
        P.n_lower[l] = (int32_t)lower[l].size(); P.n_upper[l] = (int32_t)upper[l].size();
        for (size_t r = 0; r < lower[l].size(); ++r) if (!conv_row(lower[l][r], l, P.lower[l][r])) LFAIL;
        for (size_t r = 0; r < upper[l].size(); ++r) if (!conv_row(upper[l][r], l, P.upper[l][r])) LFAIL;
    }
    if (guards.size() > TADL_MAX_ROWS) LFAIL;
    P.n_guards = (int32_t)guards.size();
    for (size_t r = 0; r < guards.size(); ++r) if (!conv_row(guards[r], 0, P.guards[r]) || guards[r].den != 1) LFAIL;
    P.n_loads = (int32_t)loads.size();
    int big = 0;
    for (size_t i = 0; i < loads.size(); ++i) {
        if (!conv_load(g.loads[loads[i]], P.loads[i])) LFAIL;
        if (g.loads[loads[i]].limit > g.loads[loads[big]].limit) big = (int)i;
    }
    std::swap(P.loads[0], P.loads[big]);                     // (order is free in a product)
    P.n_scale = (int32_t)sloads.size();
    for (size_t i = 0; i < sloads.size(); ++i) {
        if (!conv_load(g.loads[sloads[i]], P.scale[i]) || P.scale[i].cz[0] || P.scale[i].cz[1]) LFAIL;
    }
    P.cterm = cterm; P.cscale = cscale;
    double outputs = 1;
    for (int v = 0; v < g.n_outer; ++v) {
        P.outer_lo[v] = prog.outer_lo[v]; P.outer_ext[v] = prog.outer_ext[v]; P.out_coef[v] = prog.out_coef[v];
        const uint64_t d = (uint64_t)std::max(1, prog.outer_ext[v]);
        int s = 0; while ((uint64_t(1) << s) < d) ++s;
        P.div_mul[v] = (uint32_t)(((uint64_t(1) << (31 + s)) / d) + 1);
        P.div_shift[v] = 31 + s;
        outputs *= (double)d;
    }
    P.out_base = prog.out_base; P.out_limit = prog.out_limit; P.accumulate = prog.accumulate;
    // ---- which way the lanes run: along an outer variable that makes the largest operand consecutive, else along
    //      the inner loop if that does (a warp per output), else along the longest outer variable ----
    const TadlLoad &B = P.loads[0];
    const int l_in = g.kappa - 1;
    int lane = -1;
    for (int v = 0; v < g.n_outer; ++v)
        if (std::abs(B.coef[v]) == 1 && prog.outer_ext[v] >= 32 && (lane < 0 || prog.outer_ext[v] > prog.outer_ext[lane])) lane = v;
    P.mode = 0;
    if (lane < 0 && std::abs(B.cz[l_in]) == 1 && g.vars[z_id[l_in]].ext >= 64) {
        P.mode = 1;
        lane = 0;
        for (int v = 0; v < g.n_outer; ++v) if (prog.out_coef[v] != 0 && (prog.out_coef[lane] == 0 || std::abs(prog.out_coef[v]) < std::abs(prog.out_coef[lane]))) lane = v;
    }
    if (lane < 0) { lane = 0; for (int v = 0; v < g.n_outer; ++v) if (prog.outer_ext[v] > prog.outer_ext[lane]) lane = v; }
    P.lane_var = lane;
    // ---- few outputs: the outermost range is shared out ----
    P.zsplit = 1;
    int64_t cells = 1;
    for (int v = g.n_outer - 1; v >= 0; --v) { P.part_coef[v] = to_i32(cells); cells = mul_ck(cells, prog.outer_ext[v]); }
    P.part_limit = to_i32(cells);
    const double ext0 = (double)std::max<int64_t>(1, g.vars[z_id[0]].ext);
    const double want = P.mode == 1 ? 148.0 * 64 : 148.0 * 2048;          // warps / threads that fill the GPU
    if (allow_split && outputs < want / 2 && cells <= (1 << 22)) {
        double s = std::ceil(want / outputs);
        // every share keeps enough terms: eight of a single loop (128 when a warp walks it), a whole run of the inner loop
        s = std::min(s, std::max(1.0, std::floor(ext0 / (g.kappa == 2 ? 1.0 : P.mode == 1 ? 128.0 : 8.0))));
        s = std::min(s, 1024.0);
        while (s > 1 && (s + 1) * (double)cells > (double)(1 << 25)) s -= 1;
        P.zsplit = (int32_t)std::max(1.0, s);
    }
    // a masked gradient's box also holds positions that are no elements (their offsets may fall on real ones): the
    // reduction writes only where the guards held
    P.live_plane = (P.zsplit > 1 && prog.write_only_live) ? 1 : 0;
    if (P.zsplit <= 1) prog.write_only_live = 0;
    k.line = {P};
    k.vec = 0; k.vec_u = 0;
    prog.zsplit = P.zsplit; prog.part_limit = P.part_limit; prog.n_outer = g.n_outer;
    for (int v = 0; v < g.n_outer; ++v) prog.part_coef[v] = P.part_coef[v];
    char line[256];
    std::snprintf(line, sizeof line, "; line sums: %d loads x %d loops, outer factor of %d loads, %s, lanes along variable %d, %d shares, %d guards\n",
                  P.n_loads, P.n_loops, P.n_scale, P.mode == 1 ? "a warp per output" : "a thread per output", P.lane_var, P.zsplit, P.n_guards);
    k.listing = line;
    return true;
}

}  // namespace tad

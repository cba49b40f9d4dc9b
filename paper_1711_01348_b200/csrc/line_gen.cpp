// Recogniser for line-sum programs (line.h): a gradient kernel (one or two summation loops with the bound rows
// of Sec. 4.2) whose term is a product of index expressions and constants, with a factor outside the sums that
// is again such a product.  After the function tables of the optimisation pass most derivative terms have this
// form (df times pre-evaluated functions of the arguments), and the kernel runs them without interpretation.
#include <algorithm>
#include <climits>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>

#include "gen.h"
#define LFAIL return false

namespace tad {

bool try_line(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower_in,
              const std::vector<std::vector<TadpRow>> &upper_in, const std::vector<TadpRow> &guards)
{
    if (g.p.opt.debug_bounds || root < 0 || g.kappa > 2 || g.n_outer < 1 || g.n_outer > 4) return false;
    TadpProgram &prog = k.prog;
    // a kernel without kernel coordinates whose value is one sum with constant bounds (a short sum the optimisation
    // pass evaluates ahead of its kernel) is a line sum over that sum's variable
    int n_loops = g.kappa, sum_var = -1;
    std::vector<std::vector<TadpRow>> own_lower, own_upper;
    if (g.kappa == 0) {
        const Inst top = g.inst[root];
        if (top.op != I_SUM || top.temp >= 0 || scale >= 0 || !guards.empty() || prog.write_only_live) return false;
        if (top.lo < INT32_MIN / 2 || top.hi > INT32_MAX / 2 || top.hi < top.lo) return false;
        TadpRow lo{}, hi{};
        lo.den = hi.den = 1; lo.c0 = (int32_t)top.lo; hi.c0 = (int32_t)top.hi;
        own_lower = {{lo}}; own_upper = {{hi}};
        sum_var = top.var; n_loops = 1; root = top.a;
        // (the outer variables must be the first n_outer ones: kernels the optimisation pass builds may order them otherwise)
        if (sum_var < g.n_outer || sum_var >= TADP_MAX_VARS) return false;
        for (int v = 0; v < g.n_outer; ++v) if (g.vars[v].kind != 0) return false;
    }
    const std::vector<std::vector<TadpRow>> &lower = g.kappa == 0 ? own_lower : lower_in;
    const std::vector<std::vector<TadpRow>> &upper = g.kappa == 0 ? own_upper : upper_in;
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
    const int z_id[2] = {g.kappa == 0 ? sum_var : g.n_outer + g.zorder[0], g.kappa == 2 ? g.n_outer + g.zorder[1] : -1};
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
    P.n_outer = g.n_outer; P.n_loops = n_loops;
    for (int l = 0; l < n_loops; ++l) {
        if (lower[l].empty() || upper[l].empty() || lower[l].size() > TADL_MAX_ROWS || upper[l].size() > TADL_MAX_ROWS) LFAIL;
        P.n_lower[l] = (int32_t)lower[l].size(); P.n_upper[l] = (int32_t)upper[l].size();
        for (size_t r = 0; r < lower[l].size(); ++r) if (!conv_row(lower[l][r], l, P.lower[l][r])) LFAIL;
        for (size_t r = 0; r < upper[l].size(); ++r) if (!conv_row(upper[l][r], l, P.upper[l][r])) LFAIL;
    }
    if (guards.size() > TADL_MAX_ROWS) LFAIL;
    P.n_guards = (int32_t)guards.size();
    for (size_t r = 0; r < guards.size(); ++r) if (!conv_row(guards[r], 0, P.guards[r]) || guards[r].den != 1) LFAIL;
    // (a load that occurs twice is read once and squared)
    {
        std::vector<int> uniq, twice;
        for (int l : loads) {
            size_t at = 0;
            while (at < uniq.size() && uniq[at] != l) ++at;
            if (at == uniq.size()) { uniq.push_back(l); twice.push_back(0); }
            else if (!twice[at]) twice[at] = 1;
            else { uniq.push_back(l); twice.push_back(0); }
        }
        int big = 0;
        for (size_t i = 0; i < uniq.size(); ++i) {
            if (!conv_load(g.loads[uniq[i]], P.loads[i])) LFAIL;
            P.loads[i].sq = twice[i];
            // load 0 is the operand the kernel streams: the largest, among equals the one more variables move
            auto moving = [&](int l) { int n = 0; for (int v = 0; v < TADP_MAX_VARS; ++v) n += g.loads[l].coef[v] != 0; return n; };
            const int64_t a = g.loads[uniq[i]].limit, b = g.loads[uniq[big]].limit;
            if (a > b || (a == b && moving(uniq[i]) > moving(uniq[big]))) big = (int)i;
        }
        P.n_loads = (int32_t)uniq.size();
        std::swap(P.loads[0], P.loads[big]);                 // (order is free in a product)
    }
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
    const int l_in = n_loops - 1;
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
    // the box of every loop variable: a row bounds the range of every output, so its extreme over the outer box
    // (and over the box of loop 0 for the rows of loop 1) bounds them all
    int64_t zlo[2] = {0, 0}, zhi[2] = {0, 0};
    for (int l = 0; l < n_loops; ++l) {
        auto extreme = [&](const TadlRow &R, bool want_max) {
            int64_t v = R.c0;
            for (int o = 0; o < g.n_outer; ++o) {
                const int64_t a = (int64_t)R.coef[o] * P.outer_lo[o], b = (int64_t)R.coef[o] * (P.outer_lo[o] + std::max(1, P.outer_ext[o]) - 1);
                v += want_max ? std::max(a, b) : std::min(a, b);
            }
            if (l == 1) { const int64_t a = (int64_t)R.cz * zlo[0], b = (int64_t)R.cz * zhi[0]; v += want_max ? std::max(a, b) : std::min(a, b); }
            return v;
        };
        auto floor_div = [](int64_t a, int64_t b) { int64_t q = a / b; return (a % b != 0 && a < 0) ? q - 1 : q; };
        int64_t lo = INT64_MIN, hi = INT64_MAX;
        for (int r = 0; r < P.n_lower[l]; ++r) lo = std::max(lo, -floor_div(-extreme(P.lower[l][r], false), P.lower[l][r].den));
        for (int r = 0; r < P.n_upper[l]; ++r) hi = std::min(hi, floor_div(extreme(P.upper[l][r], true), P.upper[l][r].den));
        if (lo < INT32_MIN / 2 || hi > INT32_MAX / 2) LFAIL;
        zlo[l] = lo; zhi[l] = std::max(lo, hi);
    }
    // the longest range of every loop: hi - lo <= (an upper row) - (a lower row) for every pair of rows, an affine
    // form over the outer box (and the box of loop 0) whose maximum interval arithmetic gives
    int64_t longest[2] = {1, 1};
    for (int l = 0; l < n_loops; ++l) {
        int64_t best = zhi[l] - zlo[l] + 1;
        for (int u = 0; u < P.n_upper[l]; ++u)
            for (int r = 0; r < P.n_lower[l]; ++r) {
                const TadlRow &U = P.upper[l][u], &L = P.lower[l][r];
                // U / du - L / dl = (U * dl - L * du) / (du * dl)
                const int64_t du = U.den, dl = L.den;
                int64_t top = (int64_t)U.c0 * dl - (int64_t)L.c0 * du;
                auto add = [&](int64_t c, int64_t lo, int64_t hi) { top += std::max(c * lo, c * hi); };
                for (int o = 0; o < g.n_outer; ++o)
                    add((int64_t)U.coef[o] * dl - (int64_t)L.coef[o] * du, P.outer_lo[o], P.outer_lo[o] + std::max(1, P.outer_ext[o]) - 1);
                if (l == 1) add((int64_t)U.cz * dl - (int64_t)L.cz * du, zlo[0], zhi[0]);
                const int64_t den = du * dl;
                int64_t q = top / den; if (top % den != 0 && top < 0) --q;       // floor
                best = std::min(best, std::max<int64_t>(1, q + 1));
            }
        longest[l] = best;
    }
    P.n_share[0] = P.n_share[1] = 1;
    // ---- shares: pieces of every range, short enough that no thread walks a long chain of dependent batches and
    //      numerous enough to fill the GPU several times over ----
    const double slots = P.mode == 1 ? 148.0 * 48 : 148.0 * 1536;          // warps / threads resident at once
    const double piece = P.mode == 1 ? 1024.0 : 64.0;                       // terms of one thread (warp) per share
    const double ext_in = (double)longest[l_in], ext_out = n_loops == 2 ? (double)longest[0] : 1.0;
    if (allow_split && outputs < slots * 4 && cells <= (1 << 22)) {
        double room = std::floor((double)(1 << 25) / (double)cells) - 1;    // planes the workspace may hold
        room = std::min(room, std::max(1.0, std::floor(slots * 16 / outputs)));   // and no more threads than sixteen rounds
        room = std::min(room, 4096.0);
        // pieces of 2^k values; a range of length n that starts anywhere inside a piece touches up to ceil(n / 2^k) + 1
        // pieces, never more than the box has
        auto cut = [&](int l, double length, double box, double want_shares) {
            int shift = 0;
            while ((double)(1 << shift) * want_shares < length && shift < 30) ++shift;
            const double pieces = std::ceil(length / (double)(1 << shift)) + (length < box ? 1 : 0);
            P.chunk_shift[l] = shift;
            P.n_share[l] = (int32_t)std::max(1.0, std::min(pieces, std::ceil(box / (double)(1 << shift)) + 1));
            P.zbox_lo[l] = to_i32(zlo[l]);
        };
        const double s_in = std::min(std::ceil(ext_in / piece), std::max(1.0, room));
        if (s_in > 1) cut(l_in, ext_in, (double)(zhi[l_in] - zlo[l_in] + 1), s_in);
        if (n_loops == 2) {
            const double s_out = std::min(ext_out, std::max(1.0, std::floor(room / P.n_share[1])));
            if (s_out > 1) cut(0, ext_out, (double)(zhi[0] - zlo[0] + 1), s_out);
        }
        P.zsplit = P.n_share[0] * P.n_share[1];
    }
    // a masked gradient's box also holds positions that are no elements (their offsets may fall on real ones): the
    // reduction writes only where the guards held
    P.unroll = 4;
    P.stream = (P.mode == 1 ? std::abs(P.loads[0].cz[l_in]) == 1 : std::abs(P.loads[0].coef[P.lane_var]) == 1) ? 1 : 0;
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
    for (int i = 0; i < P.n_loads; ++i) {
        std::snprintf(line, sizeof line, ";   load %d ptr=%d base=%d coef=[%d %d %d %d] step=[%d %d]%s\n", i, P.loads[i].ptr, P.loads[i].base, P.loads[i].coef[0],
                      P.loads[i].coef[1], P.loads[i].coef[2], P.loads[i].coef[3], P.loads[i].cz[0], P.loads[i].cz[1], P.loads[i].sq ? " squared" : "");
        k.listing += line;
    }
    for (int l = 0; l < P.n_loops; ++l) {
        std::snprintf(line, sizeof line, ";   loop %d: %d lower rows, %d upper rows, first lower c0=%d den=%d, first upper c0=%d den=%d, %d pieces of 2^%d\n", l, P.n_lower[l], P.n_upper[l],
                      P.lower[l][0].c0, P.lower[l][0].den, P.upper[l][0].c0, P.upper[l][0].den, P.n_share[l], P.chunk_shift[l]);
        k.listing += line;
    }
    std::snprintf(line, sizeof line, ";   out base=%d coef=[%d %d %d %d] constant %g x %g\n", P.out_base, P.out_coef[0], P.out_coef[1], P.out_coef[2], P.out_coef[3], P.cterm, P.cscale);
    k.listing += line;
    return true;
}

}  // namespace tad

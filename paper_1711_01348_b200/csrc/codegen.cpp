// Code generator (host only): scalar reverse-mode differentiation of the expression (Sec. 2),
// sum liberation (Sec. 5.2), loop scheduling and emission of the interpreter's bytecode.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <functional>
#include <tuple>

#include "gen.h"

namespace tad {

namespace {

// ---- scheduling and emission ----------------------------------------------------------

const char *op_name(int op)
{
    static const char *names[] = {"END", "CONST", "ZERO", "LOAD", "LDT", "NEG", "SQR", "CUBE", "HSUM", "MULC", "ADDC",
                                  "LDADD", "LDMUL", "LDADDSQ", "SCALE", "FN", "STT", "ACC", "ADD", "SUB", "MUL", "DIV",
                                  "SUMADD", "SUMEND", "FMAT", "MACC", "FMA", "SLOOP", "SEND", "USLOOP", "USEND", "ZLOOP", "ZEND", "XLOOP"};
    return op < P_NUM_OPS ? names[op] : "?";
}

struct Emitter {
    Gen &g;
    std::vector<TadpInsn> code;
    std::vector<TadpLoop> loops;
    int depth = 0, max_depth = 0;
    std::vector<int> depth_at;           // operand stack depth before every word

    explicit Emitter(Gen &gen) : g(gen) {}

    // k_override >= 0: the handler number carries a loop variable instead of the stack depth
    int emit(int op, int a = 0, int b = 0, int32_t imm = 0, int delta = 0, int k_override = -1)
    {
        if (depth + delta > TADP_MAX_DEPTH - 1) throw Unsupported("expression needs a deeper operand stack");
        TadpInsn w{};
        w.handler = (uint16_t)(op * 8 + (k_override >= 0 ? k_override : depth));
        w.a = (uint8_t)a; w.b = (uint8_t)b; w.imm = imm;
        code.push_back(w);
        depth_at.push_back(depth);
        depth += delta;
        max_depth = std::max(max_depth, depth);
        if ((int)code.size() >= TADP_MAX_CODE) throw Unsupported("program longer than TADP_MAX_CODE words");
        return (int)code.size() - 1;
    }
    static int32_t fbits(float f) { int32_t b; std::memcpy(&b, &f, 4); return b; }
    std::string listing() const
    {
        std::string out;
        for (size_t i = 0; i < code.size(); ++i) {
            char line[160];
            float f; std::memcpy(&f, &code[i].imm, 4);
            std::snprintf(line, sizeof line, "%3zu  d=%d  %-7s a=%d b=%d imm=%d (%g)\n", i, depth_at[i], op_name(code[i].handler >> 3),
                          code[i].a, code[i].b, code[i].imm, (double)f);
            out += line;
        }
        return out;
    }

    bool inline_ok(int i) const { return g.inst[i].temp < 0; }
    // the value does not vary along the element variable (and is not computed inside its sum loop)
    int same_for_all_u(int i) const { return g.unroll_var >= 0 && !(g.inst[i].deps & (1u << g.unroll_var)) ? 1 : 0; }
    bool is_inline_load(int i) const { return g.inst[i].op == I_LOAD && g.inst[i].temp < 0; }

    // emits code that leaves the value of instance i on the stack
    void expr(int i)
    {
        if (g.inst[i].temp >= 0) { emit(P_LDT, g.inst[i].temp, 0, 0, +1); return; }
        body(i);
    }
    void body(int i)
    {
        const Inst in = g.inst[i];
        switch (in.op) {
        case I_CONST: emit(P_CONST, 0, 0, fbits(in.imm), +1); break;
        case I_LOAD: emit(P_LOAD, in.load, 0, 0, +1); break;
        case I_NEG: expr(in.a); emit(P_NEG); break;
        case I_EXP: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_EXP); break;
        case I_LOG: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_LOG); break;
        case I_SIN: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_SIN); break;
        case I_COS: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_COS); break;
        case I_TANH: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_TANH); break;
        case I_SINH: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_SINH); break;
        case I_COSH: expr(in.a); emit(P_FN, same_for_all_u(in.a), F_COSH); break;
        case I_SQR: {
            const Inst &ad = g.inst[in.a];
            if (ad.op == I_ADD && inline_ok(in.a) && (is_inline_load(ad.a) || is_inline_load(ad.b)) &&
                !(g.inst[ad.a].op == I_MUL && inline_ok(ad.a)) && !(g.inst[ad.b].op == I_MUL && inline_ok(ad.b))) {
                const int ld = is_inline_load(ad.b) ? ad.b : ad.a, other = is_inline_load(ad.b) ? ad.a : ad.b;
                expr(other); emit(P_LDADDSQ, g.inst[ld].load);
            } else { expr(in.a); emit(P_SQR); }
            break;
        }
        case I_POWI:
            expr(in.a);
            if (in.ipow == 3) emit(P_CUBE); else emit(P_FN, same_for_all_u(in.a), F_POWI, in.ipow);
            break;
        case I_MULC: expr(in.a); emit(P_MULC, 0, 0, fbits(in.imm)); break;
        case I_ADDC: expr(in.a); emit(P_ADDC, 0, 0, fbits(in.imm)); break;
        case I_ADD: {
            // a*b + c as one fused operation when the product is used only here
            int m = -1, o = -1;
            if (g.inst[in.a].op == I_MUL && inline_ok(in.a)) { m = in.a; o = in.b; }
            else if (g.inst[in.b].op == I_MUL && inline_ok(in.b)) { m = in.b; o = in.a; }
            if (m >= 0 && (g.inst[g.inst[m].a].temp >= 0 || g.inst[g.inst[m].b].temp >= 0)) {
                // product with a temporary: the temporary is read by the fused word itself
                const int tf = g.inst[g.inst[m].b].temp >= 0 ? g.inst[m].b : g.inst[m].a;
                const int other = tf == g.inst[m].b ? g.inst[m].a : g.inst[m].b;
                expr(other); expr(o); emit(P_FMAT, g.inst[tf].temp, 0, 0, -1);
            }
            else if (m >= 0) { expr(g.inst[m].a); expr(g.inst[m].b); expr(o); emit(P_FMA, 0, 0, 0, -2); }
            else if (is_inline_load(in.b)) { expr(in.a); emit(P_LDADD, g.inst[in.b].load); }
            else if (is_inline_load(in.a)) { expr(in.b); emit(P_LDADD, g.inst[in.a].load); }
            else { expr(in.a); expr(in.b); emit(P_ADD, 0, 0, 0, -1); }
            break;
        }
        case I_SUB: expr(in.a); expr(in.b); emit(P_SUB, 0, 0, 0, -1); break;
        case I_MUL:
            if (is_inline_load(in.b)) { expr(in.a); emit(P_LDMUL, g.inst[in.b].load); }
            else if (is_inline_load(in.a)) { expr(in.b); emit(P_LDMUL, g.inst[in.a].load); }
            else { expr(in.a); expr(in.b); emit(P_MUL, 0, 0, 0, -1); }
            break;
        case I_DIV: expr(in.a); expr(in.b); emit(P_DIV, 0, 0, 0, -1); break;
        case I_SUM: {
            TadpLoop L{};
            L.var = in.var; L.const_lo = (int32_t)in.lo; L.const_hi = (int32_t)in.hi;
            if ((int)loops.size() >= TADP_MAX_LOOPS) throw Unsupported("too many loops in one kernel");
            loops.push_back(L);
            int id = (int)loops.size() - 1;
            const bool over_elements = in.var == g.unroll_var;   // the element variable runs over this sum
            emit(P_ZERO, 0, 0, 0, +1);
            int begin = emit(over_elements ? P_USLOOP : P_SLOOP, id, 0, 0, 0, in.var);
            temps_of_sum(i);
            const Inst inner = g.inst[in.a];
            if (!over_elements && inner.op == I_SUM && inline_ok(in.a) && inner.var != g.unroll_var) {
                // a sum whose summand is a sum: the inner loop adds its summands to the same accumulator;
                // the longer of the two ranges runs innermost (the order of a sum of sums is free)
                TadpLoop L2{};
                L2.var = inner.var; L2.const_lo = (int32_t)inner.lo; L2.const_hi = (int32_t)inner.hi;
                if ((int)loops.size() >= TADP_MAX_LOOPS) throw Unsupported("too many loops in one kernel");
                int outer_var = in.var;
                if (inner.hi - inner.lo < in.hi - in.lo && swap_ok(i, in.a)) {
                    std::swap(loops[id], L2);
                    outer_var = inner.var;
                    code[begin].handler = (uint16_t)(P_SLOOP * 8 + outer_var);
                }
                loops.push_back(L2);
                const int id2 = (int)loops.size() - 1;
                const int ib = emit(P_SLOOP, id2, 0, 0, 0, loops[id2].var);
                temps_of_sum(in.a);
                expr(inner.a);
                const int ie = emit(P_SUMEND, id2, 0, ib + 1, -1);
                code[ib].imm = ie + 1;
                const int oe = emit(P_SEND, id, 0, begin + 1, 0, outer_var);
                code[begin].imm = oe + 1;
                break;
            }
            expr(in.a);
            int end;
            if (over_elements) {
                emit(P_SUMADD, 0, 0, 0, -1);
                end = emit(P_USEND, id, 0, begin + 1, 0, in.var);
            } else end = emit(P_SUMEND, id, 0, begin + 1, -1);
            if (over_elements) emit(P_HSUM);
            code[begin].imm = end + 1;
            break;
        }
        }
    }
    // nested sums that share an accumulator may trade places when no temporary belongs to either of
    // them (a temporary is evaluated at the head of its own loop)
    bool swap_ok(int outer_sum, int inner_sum) const
    {
        for (const Inst &in : g.inst)
            if (in.temp >= 0 && in.uses > 0 && (in.home_sum == inner_sum || in.home_sum == outer_sum)) return false;
        return true;
    }
    void temps_of_sum(int sum_inst)
    {
        for (int i = 0; i < (int)g.inst.size(); ++i)
            if (g.inst[i].temp >= 0 && g.inst[i].uses > 0 && g.inst[i].home_sum == sum_inst) { body(i); emit(P_STT, g.inst[i].temp, 0, 0, -1); }
    }
    void temps_of_level(int level)
    {
        for (int i = 0; i < (int)g.inst.size(); ++i)
            if (g.inst[i].temp >= 0 && g.inst[i].uses > 0 && g.inst[i].home_sum < 0 && g.inst[i].zlevel == level) { body(i); emit(P_STT, g.inst[i].temp, 0, 0, -1); }
    }
};

int64_t kernel_col_extent(const AccessPlan &ap, int col)
{
    int64_t best = INT64_MAX;
    for (int d = 0; d < ap.n; ++d) {
        int64_t k = std::llabs(ap.V(d, ap.R + col));
        if (k) best = std::min(best, (ap.box_hi[d] - ap.box_lo[d]) / k + 1);
    }
    return best == INT64_MAX ? 1 : best;
}

double inst_weight(const Inst &in)
{
    switch (in.op) {
    case I_CONST: return 0.0;
    case I_LOAD: return 2.0;
    case I_EXP: case I_LOG: case I_SIN: case I_COS: case I_TANH: case I_SINH: case I_COSH: return 8.0;
    case I_DIV: return 4.0;
    case I_POWI: return (double)std::max(1, std::abs(in.ipow) - 1);
    default: return 1.0;
    }
}

// marks use counts of everything reachable from `root`
void count_uses(Gen &g, int root, int root2 = -1)
{
    for (Inst &in : g.inst) in.uses = 0;
    std::vector<int> stack{root};
    g.inst[root].uses = 1;
    std::vector<bool> seen(g.inst.size(), false);
    seen[root] = true;
    if (root2 >= 0 && root2 != root) { stack.push_back(root2); g.inst[root2].uses += 1; seen[root2] = true; }
    while (!stack.empty()) {
        int i = stack.back(); stack.pop_back();
        for (int c : {g.inst[i].a, g.inst[i].b}) {
            if (c < 0) continue;
            g.inst[c].uses++;
            if (!seen[c]) { seen[c] = true; stack.push_back(c); }
        }
    }
}

// home of every instance for the current loop order
void place(Gen &g)
{
    std::vector<int> sum_depth(g.vars.size(), 0);
    for (Inst &in : g.inst) {
        in.zlevel = 0;
        for (int col = 0; col < g.kappa; ++col)
            if (in.deps & (1u << (g.n_outer + col))) in.zlevel = std::max(in.zlevel, g.zpos[col] + 1);
    }
    // depth of a bound sum = 1 + max depth of the bound variables its own instance depends on
    bool changed = true;
    while (changed) {
        changed = false;
        for (int v = 0; v < (int)g.vars.size(); ++v) {
            if (g.vars[v].kind != 2 || g.vars[v].sum_inst < 0) continue;
            int d = 1;
            for (int w = 0; w < (int)g.vars.size(); ++w)
                if (g.vars[w].kind == 2 && (g.inst[g.vars[v].sum_inst].deps & (1u << w))) d = std::max(d, sum_depth[w] + 1);
            if (d != sum_depth[v]) { sum_depth[v] = d; changed = true; }
        }
    }
    for (Inst &in : g.inst) {
        in.home_sum = -1;
        int best = 0;
        for (int v = 0; v < (int)g.vars.size(); ++v)
            if (g.vars[v].kind == 2 && (in.deps & (1u << v)) && sum_depth[v] > best) { best = sum_depth[v]; in.home_sum = g.vars[v].sum_inst; }
    }
}

// estimated warp-instructions for the current loop order and a lane variable
double schedule_cost(Gen &g, int root, int lane)
{
    place(g);
    double total = 0;
    for (int i = 0; i < (int)g.inst.size(); ++i) {
        const Inst &in = g.inst[i];
        if (!in.uses) continue;
        double execs = 1;
        for (int v = 0; v < g.n_outer; ++v) {
            double e = (double)g.vars[v].ext;
            if (v == lane) e = std::ceil(e / 32.0);
            execs *= e;
        }
        int level = (i == root) ? g.kappa : in.zlevel;
        if (in.home_sum >= 0) level = std::max(level, g.inst[in.home_sum].zlevel);
        for (int l = 0; l < level; ++l) {
            int v = g.n_outer + g.zorder[l];
            double e = (double)g.vars[v].ext;
            if (v == lane) e = std::ceil(e / 32.0);
            execs *= e;
        }
        for (int v = 0; v < (int)g.vars.size(); ++v)
            if (g.vars[v].kind == 2 && (in.deps & (1u << v))) execs *= (double)g.vars[v].ext;
        double w = inst_weight(in);
        if (in.op == I_LOAD) {
            int64_t cl = std::llabs((int64_t)g.loads[in.load].coef[lane]);
            double sectors = cl == 0 ? 1 : cl == 1 ? 4 : (double)std::min<int64_t>(32, 4 * cl);
            w += sectors;
        }
        total += execs * w;
    }
    return total;
}


// worst-case magnitude of a row numerator over the variable boxes must stay inside int32
void check_row_range(const TadpRow &r, const std::vector<int64_t> &vlo, const std::vector<int64_t> &vhi)
{
    int64_t mn = r.c0, mx = r.c0;
    for (int v = 0; v < TADP_MAX_VARS; ++v) {
        int64_t c = r.coef[v];
        if (!c) continue;
        mn = add_ck(mn, mul_ck(c, c > 0 ? vlo[v] : vhi[v]));
        mx = add_ck(mx, mul_ck(c, c > 0 ? vhi[v] : vlo[v]));
    }
    if (mn <= -(int64_t(1) << 30) || mx >= (int64_t(1) << 30)) throw Overflow();
}

void finish_stats(Gen &g, Kernel &k, bool backward, int64_t outputs, int64_t terms, bool zero_fill)
{
    tad_plan &p = g.p;
    KernelStats &s = k.stats;
    s.outputs = outputs; s.terms = terms;
    s.bytecode_words = k.prog.n_code; s.n_launches = 1 + (zero_fill ? 1 : 0);
    auto bindings = [&](uint32_t adeps) {
        double n = 1;
        for (int d = 0; d < p.n_out + p.n_sum; ++d)
            if (adeps & (1u << d)) n *= d < p.n_out ? (double)p.out_shape[d] : (double)(p.sum_hi[d - p.n_out] - p.sum_lo[d - p.n_out] + 1);
        for (int v = 0; v < (int)g.vars.size(); ++v)
            if (adeps & (1u << (16 + v))) n *= (double)g.vars[v].ext;
        return n;
    };
    std::map<int, double> ptr_bytes;
    for (int i = 0; i < (int)g.inst.size(); ++i) {
        const Inst &in = g.inst[i];
        if (!in.uses) continue;
        double n = bindings(in.adeps);
        switch (in.op) {
        case I_CONST: break;
        case I_LOAD: {
            const TadpLoad &L = g.loads[in.load];
            bool contiguous = false;
            for (int v = 0; v < TADP_MAX_VARS; ++v) if (std::abs(L.coef[v]) == 1) contiguous = true;
            double bytes = std::min(n * (contiguous ? 4.0 : 32.0), 4.0 * L.limit);
            ptr_bytes[L.ptr] = std::max(ptr_bytes[L.ptr], bytes);
            break;
        }
        case I_EXP: case I_LOG: case I_SIN: case I_COS: case I_TANH: case I_SINH: case I_COSH:
            s.alg_flops += n; s.alg_trans += n; break;
        case I_POWI: s.alg_flops += n * std::max(1, std::abs(in.ipow) - 1); break;
        case I_SUM:
            // one add per summand; a sum whose summand is a sum adds nothing of its own (they share one accumulator)
            if (g.inst[in.a].op != I_SUM) s.alg_flops += bindings(g.inst[in.a].adeps | (1u << (16 + in.var)));
            break;
        default: s.alg_flops += n; break;
        }
    }
    if (backward) s.alg_flops += (double)terms;         // the accumulation of the terms
    for (auto &kv : ptr_bytes) s.alg_bytes += kv.second;
    s.alg_bytes += 4.0 * outputs;
}

// Element variable B: a second loop variable spread over further elements of each thread.
// It pays when some load is strided across the lanes (every lane touches its own 32-byte
// sector) but contiguous along B: the thread then reads its own row with 128-bit loads and
// uses the sector in full; a strided load that does not depend on B is fetched once for all its
// elements.  Candidates: outer variables (a tile of gradient elements per thread) and bound
// sums (several summands per trip).
void choose_element_variable(Gen &g, bool allow_outer_product, uint32_t excluded = 0)
{
    g.unroll_var = -1;
    if (g.p.opt.debug_bounds) return;            // debug plans use the narrow kernels
    const int A = g.lane_var;
    double best = 0;
    for (int v = 0; v < (int)g.vars.size(); ++v) {
        if (v == A || g.vars[v].ext < 4 || g.vars[v].kind == 1 || ((excluded >> v) & 1u)) continue;
        if (g.vars[v].kind == 2 && (g.vars[v].sum_inst < 0 || !g.inst[g.vars[v].sum_inst].uses)) continue;
        double score = 0;
        bool fixes_strided = false;
        bool lane_free_load = false, u_free_load = false;   // a load that varies with v only, one that varies with A only
        bool shared_stream = false, own_stream = false;     // loads inside the summation loops: the same for every u, one per u
        for (const Inst &in : g.inst) {
            if (!in.uses || in.op != I_LOAD) continue;
            const TadpLoad &L = g.loads[in.load];
            const int64_t ca = std::llabs((int64_t)L.coef[A]), cb = std::llabs((int64_t)L.coef[v]);
            // weight: how often the load runs (loads inside bound sums and inner loops dominate)
            double w = 1;
            for (int x = g.n_outer; x < (int)g.vars.size(); ++x)
                if (x != v && (in.deps & (1u << x))) w *= (double)g.vars[x].ext;
            if (cb != 0 && ca == 0) lane_free_load = true;
            if (cb == 0 && ca != 0) u_free_load = true;
            if (w > 1 && cb == 0) shared_stream = true;
            if (w > 1 && cb != 0) own_stream = true;
            if (cb == 1 && ca >= 8) { score += 4 * w; fixes_strided = true; }          // strided load becomes row reads
            else if (cb == 0 && ca >= 8) { score += 3 * w; fixes_strided = true; }     // strided load shared by all u
            else if (cb == 0) score += w;
            else if (cb == 1 && ca == 0) score += 0.5 * w;
        }
        // outer-product structure: one load per value of v and one per value of A serve UB x TA elements
        const bool outer_product = allow_outer_product && lane_free_load && u_free_load && g.vars[v].ext >= 8;
        // a summation that streams one tensor for every output and another that UB outputs can share: a tile of
        // outputs per thread reads the shared one once (less traffic from L2 and HBM per term)
        const bool shared_reads = allow_outer_product && g.kappa >= 1 && g.vars[v].kind == 0 && shared_stream && own_stream &&
                                  g.vars[v].ext >= 8;
        if ((fixes_strided || outer_product || shared_reads) && score > best) { best = score; g.unroll_var = v; }
    }
}

// ---- fused innermost loops ----------------------------------------------------------------
// An innermost loop whose body is a short chain of loads and arithmetic on at most two live values
// (plus two loop-invariant ones) is rewritten as an accumulator program (TadpBody) and the body
// and loop end are replaced by one P_XLOOP word: the interpreter then runs every trip of the loop
// without fetching and dispatching a word per operation.  Everything else keeps the general form.
struct BodyDraft {
    std::vector<uint8_t> steps;
    std::vector<int> loads;
    std::vector<std::pair<int, int32_t>> inv;   // (kind, value)
    int term = 0;
    bool uses_y = false;
};

bool draft_body(const std::vector<TadpInsn> &code, int first, int last, int term_op, BodyDraft &d)
{
    int vd = 0;   // live values of the body: 0, 1 (X) or 2 (Y below X)
    auto inv_slot = [&](int kind, int32_t value) {
        for (size_t q = 0; q < d.inv.size(); ++q) if (d.inv[q].first == kind && d.inv[q].second == value) return (int)q;
        if (d.inv.size() >= 2) return -1;
        d.inv.push_back({kind, value});
        return (int)d.inv.size() - 1;
    };
    auto load_step = [&](int id, int cmb) {
        int j = -1;
        for (size_t q = 0; q < d.loads.size(); ++q) if (d.loads[q] == id) j = (int)q;
        if (j < 0) { if ((int)d.loads.size() >= TADP_BODY_LOADS) return false; d.loads.push_back(id); j = (int)d.loads.size() - 1; }
        d.steps.push_back((uint8_t)(0x80 | (cmb << 2) | j));
        return true;
    };
    for (int w = first; w <= last; ++w) {
        const int op = code[w].handler >> 3;
        switch (op) {
        case P_LOAD:
            if (vd == 2) return false;
            if (vd == 1) { d.steps.push_back(BS_PUSH); d.uses_y = true; }
            if (!load_step(code[w].a, 0)) return false;
            ++vd;
            break;
        case P_LDT: case P_CONST: {
            const int q = inv_slot(op == P_LDT ? 2 : 1, op == P_LDT ? (int32_t)code[w].a : code[w].imm);
            if (q < 0 || vd == 2) return false;
            if (vd == 0) { d.steps.push_back((uint8_t)(q ? BS_LDI1 : BS_LDI0)); vd = 1; break; }
            const int next = w + 1 <= last ? code[w + 1].handler >> 3 : -1;
            if (next == P_MUL) { d.steps.push_back((uint8_t)(q ? BS_MULI1 : BS_MULI0)); ++w; }
            else if (next == P_ADD) { d.steps.push_back((uint8_t)(q ? BS_ADDI1 : BS_ADDI0)); ++w; }
            else { d.steps.push_back(BS_PUSH); d.uses_y = true; d.steps.push_back((uint8_t)(q ? BS_LDI1 : BS_LDI0)); vd = 2; }
            break;
        }
        case P_LDADD: case P_LDMUL: case P_LDADDSQ:
            if (vd < 1 || !load_step(code[w].a, op == P_LDADD ? 1 : op == P_LDMUL ? 2 : 3)) return false;
            break;
        case P_NEG: if (vd < 1) return false; d.steps.push_back(BS_NEG); break;
        case P_SQR: if (vd < 1) return false; d.steps.push_back(BS_SQR); break;
        case P_CUBE: if (vd < 1) return false; d.steps.push_back(BS_CUBE); break;
        case P_MULC: case P_ADDC: {
            const int q = inv_slot(1, code[w].imm);
            if (q < 0 || vd < 1) return false;
            d.steps.push_back((uint8_t)(op == P_MULC ? (q ? BS_MULI1 : BS_MULI0) : (q ? BS_ADDI1 : BS_ADDI0)));
            break;
        }
        case P_ADD: case P_SUB: case P_MUL: case P_DIV:
            if (vd != 2) return false;
            d.steps.push_back((uint8_t)(op == P_ADD ? BS_ADDY : op == P_SUB ? BS_SUBY : op == P_MUL ? BS_MULY : BS_DIVY));
            vd = 1;
            break;
        case P_FMAT: {
            const int q = inv_slot(2, code[w].a);
            if (q < 0 || vd != 2) return false;
            d.steps.push_back((uint8_t)(q ? BS_FMAYI1 : BS_FMAYI0));
            vd = 1;
            break;
        }
        default: return false;
        }
    }
    if (term_op == P_MACC) { if (vd != 2) return false; d.term = 1; d.uses_y = true; }
    else if (vd != 1) return false;
    return !d.steps.empty() && (int)d.steps.size() <= TADP_BODY_STEPS;
}

// returns the deepest operand stack the remaining words need
int fuse_inner_loops(Emitter &em, std::vector<TadpBody> &bodies, int depth_limit)
{
    std::vector<TadpInsn> &code = em.code;
    for (int b = 0; b < (int)code.size(); ++b) {
        const int bop = code[b].handler >> 3;
        if (bop != P_SLOOP && bop != P_USLOOP && bop != P_ZLOOP) continue;
        if ((int)bodies.size() >= TADP_MAX_BODIES) break;
        const int e = code[b].imm - 1;                       // the loop end word
        if (e <= b + 1 || e >= (int)code.size()) continue;
        const int eop = code[e].handler >> 3;
        bool innermost = true;
        for (int w = b + 1; w < e; ++w) {
            const int op = code[w].handler >> 3;
            if (op >= P_SLOOP && op <= P_XLOOP) innermost = false;
        }
        if (!innermost) continue;
        const TadpLoop &L = em.loops[code[b].a];
        int last, term_op, kind, xi;
        if (bop == P_SLOOP && eop == P_SUMEND) { last = e - 1; term_op = P_SUMEND; kind = BL_SUM; xi = 1; }
        else if (bop == P_USLOOP && eop == P_USEND && (code[e - 1].handler >> 3) == P_SUMADD) { last = e - 2; term_op = P_SUMADD; kind = BL_USUM; xi = 1; }
        else if (bop == P_ZLOOP && eop == P_ZEND && ((code[e - 1].handler >> 3) == P_ACC || (code[e - 1].handler >> 3) == P_MACC)) {
            if (L.is_relative) continue;
            last = e - 2; term_op = code[e - 1].handler >> 3; xi = 0;
            kind = L.is_lane ? BL_Z_LANE : L.depends_on_lane ? BL_Z_MASKED : BL_Z;
        } else continue;
        if (em.depth_at[b + 1] != xi) continue;             // the sum accumulator must be the bottom of the stack
        BodyDraft d;
        if (!draft_body(code, b + 1, last, term_op, d)) continue;
        if (xi + (d.uses_y ? 2 : 1) + (int)d.inv.size() > depth_limit) continue;
        TadpBody B{};
        for (size_t i = 0; i < d.steps.size(); ++i) B.steps[i] = d.steps[i];
        for (size_t i = 0; i < d.loads.size(); ++i) B.load[i] = (uint8_t)d.loads[i];
        B.n_loads = (int32_t)d.loads.size();
        B.loop_kind = kind; B.term = d.term;
        for (size_t q = 0; q < d.inv.size(); ++q) { B.inv_kind[q] = d.inv[q].first; B.inv_value[q] = d.inv[q].second; }
        // the term is the product of two loads and nothing else
        if (d.inv.empty() && d.loads.size() == 2 &&
            ((d.term == 0 && d.steps == std::vector<uint8_t>{0x80 | 0, 0x80 | (2 << 2) | 1}) ||
             (d.term == 1 && d.steps == std::vector<uint8_t>{0x80 | 0, BS_PUSH, 0x80 | 1})))
            B.dot = 1;
        bodies.push_back(B);
        // body and loop end become one word; jump targets behind it move up
        const int removed = e - (b + 1);
        TadpInsn x{};
        x.handler = (uint16_t)(P_XLOOP * 8 + xi); x.a = code[b].a; x.imm = (int32_t)bodies.size() - 1;
        code[b + 1] = x;
        code.erase(code.begin() + b + 2, code.begin() + e + 1);
        em.depth_at.erase(em.depth_at.begin() + b + 2, em.depth_at.begin() + e + 1);
        for (TadpInsn &w : code) {
            const int op = w.handler >> 3;
            const bool jumps = op == P_SLOOP || op == P_SEND || op == P_USLOOP || op == P_USEND || op == P_ZLOOP || op == P_ZEND || op == P_SUMEND;
            if (jumps && w.imm > e) w.imm -= removed;
        }
    }
    int deepest = 0;
    for (size_t i = 0; i < code.size(); ++i) {
        const int op = code[i].handler >> 3;
        if (op >= P_SLOOP && op <= P_ZEND) continue;
        int after = em.depth_at[i];
        if (op == P_XLOOP) continue;                      // checked against depth_limit when it was made
        if (op == P_CONST || op == P_ZERO || op == P_LOAD || op == P_LDT) after += 1;
        deepest = std::max(deepest, after);
    }
    return deepest;
}

// how a fused body fetches a load, given the vector shape
int body_fetch_kind(const TadpLoad &L, int ta, int ub)
{
    const bool lane_fixed = L.lane_step == 0, u_fixed = ub == 1 || L.unroll_step == 0;
    if (lane_fixed && u_fixed) return BF_ONE;
    if (ub > 1 && u_fixed) return BF_PER_T;
    if (ub > 1 && ta > 1 && lane_fixed) return BF_PER_U;
    if (ub > 1 && ub % 4 == 0 && L.unroll_step == 1) return BF_ROW;
    return BF_EACH;
}

// A program without loops and temporaries whose pending values never exceed two becomes an element-wise program
// (ew.h); a thread owns four consecutive values of the lane variable.
// Steps of an element-wise program read off the expression itself, the operand that needs the second value register
// evaluated first (so that a * (b * c + d) needs no more than X and Y whatever the order it was written in).
// need(i): value registers the evaluation of i occupies; a binary operation whose operands are both compound puts the
// first into Y, which the second must then leave alone (need 1).
bool elementwise_steps_of(const Gen &g, int root, std::vector<TadeStep> &steps)
{
    auto push_step = [&](int op, int a = 0, int b = 0, float imm = 0.f) { TadeStep s{}; s.op = (uint8_t)op; s.a = (int16_t)a; s.b = (uint8_t)b; s.imm = imm; steps.push_back(s); };
    auto is_load = [&](int i) { return g.inst[i].op == I_LOAD; };
    std::function<int(int)> need = [&](int i) -> int {
        const Inst &in = g.inst[i];
        switch (in.op) {
        case I_CONST: case I_LOAD: return 1;
        case I_SUM: return 99;
        case I_ADD: case I_MUL:
            if (is_load(in.a)) return need(in.b);
            if (is_load(in.b)) return need(in.a);
            return std::max(std::max(need(in.a), need(in.b)), std::min(need(in.a), need(in.b)) + 1);
        case I_SUB: case I_DIV: return std::max(need(in.a), need(in.b) + 1);
        default: return need(in.a);
        }
    };
    std::function<bool(int)> emit = [&](int i) -> bool {
        const Inst &in = g.inst[i];
        if (in.temp >= 0) return false;
        auto fn = [&](int f, int e = 0) { if (!emit(in.a)) return false; push_step(E_FN, e, f); return true; };
        switch (in.op) {
        case I_CONST: push_step(E_CONST, 0, 0, in.imm); return true;
        case I_LOAD: push_step(E_LD, in.load, 0); return true;
        case I_NEG: if (!emit(in.a)) return false; push_step(E_NEG); return true;
        case I_SQR: if (!emit(in.a)) return false; push_step(E_SQR); return true;
        case I_MULC: if (!emit(in.a)) return false; push_step(E_MULC, 0, 0, in.imm); return true;
        case I_ADDC: if (!emit(in.a)) return false; push_step(E_ADDC, 0, 0, in.imm); return true;
        case I_POWI:
            if (in.ipow == 3) { if (!emit(in.a)) return false; push_step(E_CUBE); return true; }
            return fn(F_POWI, in.ipow);
        case I_EXP: return fn(F_EXP);
        case I_LOG: return fn(F_LOG);
        case I_SIN: return fn(F_SIN);
        case I_COS: return fn(F_COS);
        case I_TANH: return fn(F_TANH);
        case I_SINH: return fn(F_SINH);
        case I_COSH: return fn(F_COSH);
        case I_ADD: case I_MUL: {
            const int mode = in.op == I_ADD ? 1 : 2;
            if (is_load(in.b) && !(is_load(in.a) && need(in.b) < need(in.a))) { if (!emit(in.a)) return false; push_step(E_LD, g.inst[in.b].load, mode); return true; }
            if (is_load(in.a)) { if (!emit(in.b)) return false; push_step(E_LD, g.inst[in.a].load, mode); return true; }
            const int first = need(in.a) >= need(in.b) ? in.a : in.b, second = first == in.a ? in.b : in.a;
            if (need(first) > 2 || need(second) != 1) return false;
            if (!emit(first)) return false;
            push_step(E_PUSH);
            if (!emit(second)) return false;
            push_step(in.op == I_ADD ? E_ADDY : E_MULY);
            return true;
        }
        case I_SUB: case I_DIV:
            if (need(in.a) > 2 || need(in.b) != 1) return false;
            if (!emit(in.a)) return false;
            push_step(E_PUSH);
            if (!emit(in.b)) return false;
            push_step(in.op == I_SUB ? E_SUBY : E_DIVY);
            return true;
        default: return false;
        }
    };
    if (need(root) > 2) return false;
    return emit(root) && (int)steps.size() <= TADE_MAX_STEPS;
}

bool try_elementwise(Gen &g, Kernel &k, const Emitter &em, const std::vector<TadpRow> &guards, int root)
{
    const TadpProgram &prog = k.prog;
    // (elements that a guard or a mask excludes are not evaluated by the interpreter: such kernels stay there)
    // (without guards and kernel coordinates every position of a masked gradient's box is an element)
    if (g.kappa != 0 || g.p.opt.debug_bounds || !guards.empty()) return false;
    if (g.lane_var < 0 || g.lane_var >= g.n_outer) return false;
    if ((int)g.loads.size() > TADE_MAX_LOADS) return false;
    const std::vector<TadpInsn> &code = em.code;
    const int n = (int)code.size();
    if (n < 3 || (code[n - 1].handler >> 3) != P_END) return false;
    const int term_op = code[n - 2].handler >> 3;
    if (term_op != P_ACC && term_op != P_MACC) return false;
    std::vector<TadeStep> steps;
    auto push_step = [&](int op, int a = 0, int b = 0, float imm = 0.f) { TadeStep s{}; s.op = (uint8_t)op; s.a = (int16_t)a; s.b = (uint8_t)b; s.imm = imm; steps.push_back(s); };
    const bool from_expression = root >= 0 && elementwise_steps_of(g, root, steps);
    if (!from_expression) steps.clear();
    int vd = 0;                                  // pending values: 0, 1 (X) or 2 (Y below X)
    for (int w = 0; !from_expression && w < n - 2; ++w) {
        const TadpInsn &in = code[w];
        const int op = in.handler >> 3;
        float imm; std::memcpy(&imm, &in.imm, 4);
        switch (op) {
        case P_LOAD: case P_CONST:
            if (vd == 2) return false;
            if (vd == 1) push_step(E_PUSH);
            if (op == P_LOAD) push_step(E_LD, in.a, 0); else push_step(E_CONST, 0, 0, imm);
            ++vd;
            break;
        case P_LDADD: if (vd < 1) return false; push_step(E_LD, in.a, 1); break;
        case P_LDMUL: if (vd < 1) return false; push_step(E_LD, in.a, 2); break;
        case P_LDADDSQ: if (vd < 1) return false; push_step(E_LD, in.a, 3); break;
        case P_NEG: if (vd < 1) return false; push_step(E_NEG); break;
        case P_SQR: if (vd < 1) return false; push_step(E_SQR); break;
        case P_CUBE: if (vd < 1) return false; push_step(E_CUBE); break;
        case P_MULC: if (vd < 1) return false; push_step(E_MULC, 0, 0, imm); break;
        case P_ADDC: if (vd < 1) return false; push_step(E_ADDC, 0, 0, imm); break;
        case P_FN: if (vd < 1) return false; push_step(E_FN, in.imm, in.b); break;
        case P_ADD: case P_SUB: case P_MUL: case P_DIV:
            if (vd != 2) return false;
            push_step(op == P_ADD ? E_ADDY : op == P_SUB ? E_SUBY : op == P_MUL ? E_MULY : E_DIVY);
            vd = 1;
            break;
        default: return false;
        }
    }
    if (from_expression) {}
    else if (term_op == P_MACC) { if (vd != 2) return false; push_step(E_MULY); }
    else if (vd != 1) return false;
    if ((int)steps.size() > TADE_MAX_STEPS) return false;
    // every offset the kernel can form must lie inside its tensor (interval check over the outer box)
    auto inside = [&](const int32_t *coef, int64_t base, int64_t limit) {
        int64_t lo = base, hi = base;
        for (int v = 0; v < g.n_outer; ++v) {
            const int64_t a = (int64_t)coef[v] * prog.outer_lo[v], b = (int64_t)coef[v] * (prog.outer_lo[v] + std::max(1, prog.outer_ext[v]) - 1);
            lo += std::min(a, b); hi += std::max(a, b);
        }
        return lo >= 0 && hi < limit;
    };
    for (const TadeStep &s : steps)
        if (s.op == E_LD && !inside(g.loads[s.a].coef, g.loads[s.a].base, g.loads[s.a].limit)) return false;
    if (!inside(prog.out_coef, prog.out_base, prog.out_limit)) return false;
    TadeProgram E{};
    E.n_outer = g.n_outer; E.lane_var = g.lane_var;
    for (int v = 0; v < g.n_outer; ++v) {
        E.outer_lo[v] = prog.outer_lo[v]; E.outer_ext[v] = prog.outer_ext[v]; E.out_coef[v] = prog.out_coef[v];
        // n / d = (n * mul) >> (31 + s) for n < 2^31 with s = ceil(log2 d), mul = floor(2^(31 + s) / d) + 1
        const uint64_t d = (uint64_t)std::max(1, prog.outer_ext[v]);
        int s = 0; while ((uint64_t(1) << s) < d) ++s;
        E.div_mul[v] = (uint32_t)(((uint64_t(1) << (31 + s)) / d) + 1);
        E.div_shift[v] = 31 + s;
    }
    E.out_base = prog.out_base; E.out_limit = prog.out_limit; E.accumulate = prog.accumulate;
    E.n_loads = (int32_t)g.loads.size();
    for (size_t i = 0; i < g.loads.size(); ++i) E.loads[i] = g.loads[i];
    E.n_steps = (int32_t)steps.size();
    std::copy(steps.begin(), steps.end(), E.steps);
    k.ew = {E};
    k.vec = 0; k.vec_u = 0;
    char line[200];
    std::snprintf(line, sizeof line, "; element-wise program: %d steps, %d loads, rows of %d along variable %d\n", E.n_steps, E.n_loads,
                  E.outer_ext[E.lane_var], E.lane_var);
    k.listing = line + em.listing();
    for (int i = 0; i < E.n_loads; ++i) {
        std::string t;
        for (int v = 0; v < g.n_outer; ++v) t += " " + std::to_string(E.loads[i].coef[v]);
        std::snprintf(line, sizeof line, "; load %d ptr=%d base=%d coef=[%s ]\n", i, E.loads[i].ptr, E.loads[i].base, t.c_str());
        k.listing += line;
    }
    return true;
}

// shared tail: choose temps, emit, fill the program
void emit_kernel(Gen &g, Kernel &k, int root, const std::vector<std::vector<TadpRow>> &lower,
                 const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards, bool allow_split = false,
                 bool may_factor = true)
{
    TadpProgram &prog = k.prog;
    place(g);
    // Factors of the term that no kernel coordinate touches (and constant factors) multiply the
    // finished sum once instead of every term:  sum_z (c * X * Y(z)) = c * X * sum_z Y(z).
    int scale = -1;
    if (g.kappa >= 1) {
        std::vector<int> outer_factors, inner_factors;
        float cfac = 1.f;
        std::vector<int> todo{root};
        while (!todo.empty()) {
            const int i = todo.back(); todo.pop_back();
            const Inst in = g.inst[i];
            const bool sole = i == root || in.uses == 1;
            if (in.op == I_MUL && sole) { todo.push_back(in.a); todo.push_back(in.b); }
            else if (in.op == I_MULC && sole) { cfac *= in.imm; todo.push_back(in.a); }
            else if (in.op == I_NEG && sole) { cfac = -cfac; todo.push_back(in.a); }
            else if (in.op == I_SQR && sole && g.inst[in.a].zlevel == 0 && g.inst[in.a].home_sum < 0) outer_factors.push_back(i);
            else if (in.zlevel == 0 && in.home_sum < 0 && in.op != I_CONST) outer_factors.push_back(i);
            else inner_factors.push_back(i);
        }
        if (!inner_factors.empty() && (!outer_factors.empty() || cfac != 1.f)) {
            std::sort(inner_factors.begin(), inner_factors.end());
            std::sort(outer_factors.begin(), outer_factors.end());
            int term = inner_factors[0];
            for (size_t f = 1; f < inner_factors.size(); ++f) term = g.bin(I_MUL, term, inner_factors[f]);
            if (outer_factors.empty()) scale = g.konst(cfac);
            else {
                scale = outer_factors[0];
                for (size_t f = 1; f < outer_factors.size(); ++f) scale = g.bin(I_MUL, scale, outer_factors[f]);
                scale = g.mulc(scale, cfac);
            }
            root = term;
            count_uses(g, root, scale);
            place(g);
        }
    }
    // a product of two index expressions under summations runs on the tile kernel, not in the interpreter
    if (try_contraction(g, k, root, scale, allow_split, lower, upper, guards)) return;
    // sums that can be pushed inside the term (Sec. 6's missing clean-up step): auxiliary kernels + a smaller kernel
    if (may_factor && try_factoring(g, k, root, scale, allow_split, lower, upper, guards)) return;
    // sums of products of index expressions (most derivative terms once the functions are tabulated)
    if (try_line(g, k, root, scale, allow_split, lower, upper, guards)) return;
    // a short loop whose range shifts from lane to lane will be walked relative to every element's own
    // start, which needs the elements of a thread to lie along the lane variable only
    bool relative_candidate = false;
    for (int l = 0; l < g.kappa; ++l) {
        const int v = g.n_outer + g.zorder[l];
        if (v == g.lane_var || g.vars[v].ext > 16) continue;
        for (const TadpRow &r : lower[l]) if (r.coef[g.lane_var]) relative_candidate = true;
        for (const TadpRow &r : upper[l]) if (r.coef[g.lane_var]) relative_candidate = true;
    }
    // the loop over the lane variable takes one range for the whole thread: a variable that its bounds
    // depend on cannot give the thread's elements different values
    uint32_t lane_bound_vars = 0;
    for (int l = 0; l < g.kappa; ++l) {
        if (g.n_outer + g.zorder[l] != g.lane_var) continue;
        for (const std::vector<TadpRow> *rows : {&lower[l], &upper[l]})
            for (const TadpRow &r : *rows)
                for (int x = 0; x < (int)g.vars.size(); ++x) if (r.coef[x]) lane_bound_vars |= 1u << x;
    }
    choose_element_variable(g, !relative_candidate, lane_bound_vars);
    // temporaries: shared values and values hoisted out of the loop that consumes them
    std::vector<bool> hoisted(g.inst.size(), false);
    auto effective_level = [&](int i) { return i == root ? g.kappa : g.inst[i].zlevel; };
    for (int i = 0; i < (int)g.inst.size(); ++i) {
        const Inst &in = g.inst[i];
        if (!in.uses) continue;
        for (int c : {in.a, in.b}) {
            if (c < 0 || g.inst[c].op == I_CONST) continue;
            const Inst &ch = g.inst[c];
            if (in.op == I_SUM) { if (ch.home_sum != i) hoisted[c] = true; }   // a sum's body is consumed inside its loop
            else if (ch.home_sum != in.home_sum) hoisted[c] = true;
            else if (ch.home_sum < 0 && ch.zlevel != effective_level(i)) hoisted[c] = true;
        }
    }
    int n_temps = 0;
    for (int i = 0; i < (int)g.inst.size(); ++i) {
        Inst &in = g.inst[i];
        in.temp = -1;
        if (!in.uses || in.op == I_CONST || i == root || i == scale) continue;
        if (in.uses > 1 || hoisted[i]) {
            if (n_temps >= TADP_NUM_TEMPS + TADP_MAX_SPILL) throw Unsupported("too many temporaries");
            in.temp = n_temps++;
        }
    }
    Emitter em(g);
    em.temps_of_level(0);
    std::vector<int> zbegin(g.kappa);
    for (int l = 0; l < g.kappa; ++l) {
        TadpLoop L{};
        L.var = g.n_outer + g.zorder[l];
        L.is_lane = L.var == g.lane_var;
        L.mask_level = l + 1;
        em.loops.push_back(L);
        zbegin[l] = em.emit(P_ZLOOP, (int)em.loops.size() - 1, 0, 0, 0, L.var);
        em.temps_of_level(l + 1);
    }
    if (g.inst[root].op == I_MUL && g.inst[root].temp < 0) {
        em.expr(g.inst[root].a); em.expr(g.inst[root].b);
        em.emit(P_MACC, 0, 0, 0, -2);
    } else {
        em.expr(root);
        em.emit(P_ACC, 0, 0, 0, -1);
    }
    for (int l = g.kappa - 1; l >= 0; --l) {
        int loop_id = em.code[zbegin[l]].a;
        int end = em.emit(P_ZEND, loop_id, 0, zbegin[l] + 1, 0, em.loops[loop_id].var);
        em.code[zbegin[l]].imm = end + 1;
    }
    if (scale >= 0) { em.expr(scale); em.emit(P_SCALE, 0, 0, 0, -1); }
    em.emit(P_END);
    if (em.depth != 0) throw BadExpr("internal: unbalanced operand stack");
    if (n_temps == 0 && try_elementwise(g, k, em, guards, scale < 0 ? root : -1)) return;
    // rows
    std::vector<TadpRow> rows;
    for (TadpLoop &L : em.loops) {
        if (g.vars[L.var].kind != 1) continue;
        int zl = g.zpos[L.var - g.n_outer];
        L.lower0 = (int16_t)rows.size(); L.n_lower = (int16_t)lower[zl].size();
        for (const TadpRow &r : lower[zl]) rows.push_back(r);
        L.upper0 = (int16_t)rows.size(); L.n_upper = (int16_t)upper[zl].size();
        for (const TadpRow &r : upper[zl]) rows.push_back(r);
        L.depends_on_lane = 0;
        for (int r = L.lower0; r < L.upper0 + L.n_upper; ++r)
            if (rows[r].coef[g.lane_var] || (g.unroll_var >= 0 && rows[r].coef[g.unroll_var])) L.depends_on_lane = 1;
    }
    prog.guard0 = (int32_t)rows.size(); prog.n_guards = (int32_t)guards.size();
    for (const TadpRow &r : guards) rows.push_back(r);
    if ((int)rows.size() > TADP_MAX_ROWS) throw Unsupported("too many bound rows in one kernel");
    prog.n_loads = (int32_t)g.loads.size();
    std::copy(g.loads.begin(), g.loads.end(), prog.loads);
    // relative loop: a kernel-coordinate loop whose range is short but starts at a different value
    // for every lane (the taps of a strided convolution's transpose): walking the union of all
    // lanes' ranges would leave almost every element idle
    prog.rel_var = -1;
    for (int li = (int)em.loops.size() - 1; li >= 0; --li) {
        TadpLoop &L = em.loops[li];
        if (g.unroll_var >= 0) break;
        if (g.vars[L.var].kind != 1 || L.is_lane || !L.depends_on_lane) continue;
        if (g.vars[L.var].ext > 16) continue;
        // no other loop's bounds may read this variable through a warp-uniform path
        bool inner_reads = false;
        for (const TadpLoop &M : em.loops)
            if (&M != &L && g.vars[M.var].kind == 1)
                for (int r = M.lower0; r < M.upper0 + M.n_upper; ++r) if (rows[r].coef[L.var] && !M.depends_on_lane) inner_reads = true;
        if (inner_reads) continue;
        L.is_relative = 1; prog.rel_var = L.var;
        break;
    }
    for (int i = 0; i < prog.n_loads; ++i) {
        prog.loads[i].lane_step = to_i32(32 * (int64_t)prog.loads[i].coef[g.lane_var]);
        prog.loads[i].rel_step = prog.rel_var >= 0 ? prog.loads[i].coef[prog.rel_var] : 0;
        prog.loads[i].unroll_step = g.unroll_var >= 0 ? prog.loads[i].coef[g.unroll_var] : 0;
    }
    prog.n_loops = (int32_t)em.loops.size();
    std::copy(em.loops.begin(), em.loops.end(), prog.loops);
    prog.n_rows = (int32_t)rows.size();
    std::copy(rows.begin(), rows.end(), prog.rows);
    prog.n_outer = g.n_outer;
    prog.lane_var = g.lane_var;
    prog.unroll_var = g.unroll_var;
    prog.unroll_kind = g.unroll_var < 0 ? 0 : g.unroll_var < g.n_outer ? 1 : 3;
    // Vector width and summation split.  Wide vectors amortise the interpreter's dispatch cost,
    // but only while enough warps remain to fill the GPU; when even the narrowest shape leaves
    // too few, the outermost kernel-coordinate loop is divided among several warps per output,
    // each writing a partial sum that a second launch adds up in a fixed order.
    const int64_t lane_ext = g.vars[g.lane_var].ext;
    const double target_warps = 148.0 * 16.0 * 2.0;
    const int64_t uext = g.unroll_var >= 0 ? g.vars[g.unroll_var].ext : 1;
    const bool debug = g.p.opt.debug_bounds != 0;
    // fused inner loops leave the operand stack to the rest of the program: try them with the
    // 4-deep stack of the 16-value variants first
    const bool can_fuse = !debug;
    Emitter trial(em);
    std::vector<TadpBody> bodies_wide;
    const int deepest_wide = can_fuse ? fuse_inner_loops(trial, bodies_wide, TADP_WIDE_DEPTH) : em.max_depth;
    const bool shallow = deepest_wide <= TADP_WIDE_DEPTH;
    // Product kernels: when every fused loop is a product of two loads, one of which has a value per u or
    // per t only, and the rest of the program needs a single operand slot, the thread can hold 4 x 8
    // sums (nothing but the sums has 32 entries: an outer-product or streamed multiply-add per trip).
    auto load_class = [&](const TadpLoad &L, int ta, int ub) {
        const int fk = body_fetch_kind(L, ta, ub);
        return fk == BF_ONE || fk == BF_PER_U ? 0 : fk == BF_PER_T ? 1 : 2;
    };
    bool product_only = can_fuse && g.unroll_var >= 0 && !bodies_wide.empty() && prog.rel_var < 0;
    if (product_only) {
        int deepest32 = 0;
        for (size_t i = 0; i < trial.code.size(); ++i) {
            const int op = trial.code[i].handler >> 3;
            if (op == P_XLOOP) {
                const TadpBody &B = bodies_wide[trial.code[i].imm];
                if (!B.dot || std::min(load_class(prog.loads[B.load[0]], 4, 8), load_class(prog.loads[B.load[1]], 4, 8)) > 1) product_only = false;
                deepest32 = std::max(deepest32, trial.depth_at[i]);
                continue;
            }
            if (op >= P_SLOOP && op <= P_ZEND) continue;
            int after = trial.depth_at[i];
            if (op == P_CONST || op == P_ZERO || op == P_LOAD || op == P_LDT) after += 1;
            deepest32 = std::max(deepest32, after);
        }
        if (deepest32 > 1) product_only = false;
    }
    // candidate shapes (TA, UB), widest first; 16 values per thread need the shallow stack
    struct Shape { int ta, ub; };
    std::vector<Shape> shapes;
    if (g.unroll_var >= 0 && !debug) {
        if (product_only && uext >= 8 && lane_ext >= 128) shapes.push_back({4, 8});
        if (uext >= 8 && shallow && lane_ext >= 64) shapes.push_back({2, 8});     // measured best on the intro expression
        if (uext >= 16 && shallow) shapes.push_back({1, 16});
        if (uext >= 8) shapes.push_back({1, 8});
        shapes.push_back({1, 4});
    } else {
        for (int T : {16, 8, 4, 2, 1}) {
            if (T == 16 && !shallow) continue;
            if (debug && T > 4) continue;
            if (T > 1 && lane_ext < 32 * T) continue;
            shapes.push_back({T, 1});
        }
    }
    auto items_for = [&](const Shape &sh) {
        double n = 1;
        for (int v = 0; v < g.n_outer; ++v) {
            double e = (double)prog.outer_ext[v];
            if (v == g.lane_var) e = std::ceil(e / (32.0 * sh.ta));
            else if (v == g.unroll_var) e = std::ceil(e / (double)sh.ub);
            n *= e;
        }
        return n;
    };
    prog.zsplit = 1;
    Shape pick = shapes.back();
    if (g.kappa >= 1) {
        // a summation that can be split: take the widest shape and split to fill the GPU
        pick = shapes.front();
        // compact index of an output inside a plane of partial sums: row-major over the outer box
        int64_t cells = 1;
        for (int v = g.n_outer - 1; v >= 0; --v) { prog.part_coef[v] = to_i32(cells); cells = mul_ck(cells, prog.outer_ext[v]); }
        // splitting costs a pass over zsplit planes: only when the outputs are too few to fill the GPU and every
        // output has enough terms to share out (a few dozen terms per output are summed faster than split)
        double terms_per_output = 1;
        for (int l = 0; l < g.kappa; ++l) terms_per_output *= (double)std::max<int64_t>(1, g.vars[g.n_outer + g.zorder[l]].ext);
        if (items_for(pick) < target_warps / 2 && cells <= (1 << 22) && terms_per_output >= 256) {
            TadpLoop &L0 = prog.loops[em.code[zbegin[0]].a];
            // shares of the outermost loop first; when that loop is too short, the next one is divided too
            // (share number s = s0 * S1 + s1)
            TadpLoop *L1 = g.kappa >= 2 ? &prog.loops[em.code[zbegin[1]].a] : nullptr;
            auto loop_trips = [&](const TadpLoop &L, const Shape &sh) {
                return std::max<int64_t>(1, g.vars[L.var].ext / (L.is_lane ? 32 * sh.ta : 1));
            };
            auto splits_for = [&](const Shape &sh, int64_t &S0, int64_t &S1) {
                // whole waves of resident warps (148 SMs x 16): a last wave that is mostly empty costs a full one
                const double resident = 148.0 * 16.0;
                int64_t want = (int64_t)std::ceil(2.0 * target_warps / items_for(sh));
                const double waves = std::max(1.0, std::round(items_for(sh) * (double)want / resident));
                want = std::max<int64_t>(1, (int64_t)std::floor(waves * resident / items_for(sh)));
                S0 = std::min<int64_t>(std::min<int64_t>(want, loop_trips(L0, sh)), 4096);
                S1 = 1;
                if (L1 && S0 < want) S1 = std::min<int64_t>(std::min<int64_t>((want + S0 - 1) / S0, loop_trips(*L1, sh)), std::max<int64_t>(1, 4096 / S0));
                while (S0 * S1 > 1 && (S0 * S1 + 1) * cells > (int64_t(1) << 25)) { if (S1 > 1) S1 /= 2; else S0 /= 2; }   // <= 128 MB of partial sums
                return S0 * S1;
            };
            // when the loops are too short to give the widest shape enough shares, narrower shapes bring more warps
            int64_t S0 = 1, S1 = 1;
            for (const Shape &sh : shapes) {
                pick = sh;
                if (items_for(sh) * (double)splits_for(sh, S0, S1) >= target_warps / 2) break;
            }
            const int64_t S = splits_for(pick, S0, S1);
            if (S >= 2) {
                prog.zsplit = (int32_t)S; prog.part_limit = to_i32(cells);
                if (S0 > 1) { L0.is_split = 1; L0.split_n = (int32_t)S0; L0.split_div = (int32_t)S1; }
                if (S1 > 1) { L1->is_split = 1; L1->split_n = (int32_t)S1; L1->split_div = 1; }
            }
        } else if (items_for(pick) < target_warps / 2) {
            // few outputs with short summations: the narrowest shape that fills the GPU (more warps, fewer values each)
            for (const Shape &sh : shapes) { pick = sh; if (items_for(sh) >= target_warps / 2) break; }
        }
    } else {
        // element-wise kernel: the widest shape that still leaves enough warps
        for (const Shape &sh : shapes) if (items_for(sh) >= target_warps) { pick = sh; break; }
    }
    k.vec = pick.ta; k.vec_u = pick.ub;
    std::vector<TadpBody> bodies;
    if (can_fuse) {
        if (pick.ta * pick.ub >= 16) { em.code = trial.code; em.depth_at = trial.depth_at; bodies = bodies_wide; }
        else fuse_inner_loops(em, bodies, TADP_MAX_DEPTH - 1);
    }
    for (TadpBody &B : bodies)
        for (int i = 0; i < TADP_BODY_STEPS; ++i)
            if (B.steps[i] & 0x80) B.steps[i] |= (uint8_t)(body_fetch_kind(prog.loads[B.load[B.steps[i] & 3]], pick.ta, pick.ub) << 4);
    if (pick.ta * pick.ub >= 32)
        for (TadpBody &B : bodies) {
            // P is the operand of the smaller class: its buffer is small and the other one is never stored
            if (load_class(prog.loads[B.load[1]], pick.ta, pick.ub) < load_class(prog.loads[B.load[0]], pick.ta, pick.ub)) std::swap(B.load[0], B.load[1]);
            B.dot_pclass = load_class(prog.loads[B.load[0]], pick.ta, pick.ub);
            for (int j = 0; j < 2; ++j) B.dot_fk[j] = body_fetch_kind(prog.loads[B.load[j]], pick.ta, pick.ub);
        }
    // a fused loop under per-element masks keeps a range per element besides the values: measured faster with
    // 168 registers and 12 warps per SM than with 128 and 16 (cfg4 dx 0.90 -> 0.73 ms), unlike everything else
    k.rich = false;
    if (pick.ta == 16 && pick.ub == 1 && !debug && prog.rel_var < 0)
        for (const TadpBody &B : bodies) if (B.loop_kind == BL_Z_MASKED) k.rich = true;
    prog.n_bodies = (int32_t)bodies.size();
    std::copy(bodies.begin(), bodies.end(), prog.bodies);
    prog.n_code = (int32_t)em.code.size();
    std::copy(em.code.begin(), em.code.end(), prog.code);
    char head[256];
    std::snprintf(head, sizeof head, "; vars=%zu outer=%d kappa=%d lane_var=%d unroll_var=%d vec=%dx%d%s zsplit=%d temps=%d max_depth=%d loads=%d rows=%d guards=%d\n",
                  g.vars.size(), g.n_outer, g.kappa, g.lane_var, g.unroll_var, k.vec, k.vec_u, k.rich ? "r" : "", prog.zsplit, n_temps, em.max_depth, prog.n_loads, prog.n_rows, prog.n_guards);
    k.listing = head + em.listing();
    // tables the code refers to: variables, loads, loops, bound rows
    auto coefs = [&](const int32_t *c) {
        std::string t;
        for (int v = 0; v < (int)g.vars.size() && v < TADP_MAX_VARS; ++v) { char b2[24]; std::snprintf(b2, sizeof b2, " %d", c[v]); t += b2; }
        return t;
    };
    char line[256];
    for (int v = 0; v < (int)g.vars.size(); ++v) {
        std::snprintf(line, sizeof line, "; var %d kind=%d ext=%lld\n", v, g.vars[v].kind, (long long)g.vars[v].ext);
        k.listing += line;
    }
    for (int i = 0; i < prog.n_loads; ++i) {
        std::snprintf(line, sizeof line, "; load %d ptr=%d base=%d coef=[%s ]\n", i, prog.loads[i].ptr, prog.loads[i].base, coefs(prog.loads[i].coef).c_str());
        k.listing += line;
    }
    for (int i = 0; i < prog.n_loops; ++i) {
        const TadpLoop &L = prog.loops[i];
        std::snprintf(line, sizeof line, "; loop %d var=%d lane=%d split=%d relative=%d lane_dependent=%d const=[%d,%d] lower=%d+%d upper=%d+%d\n", i, L.var, L.is_lane,
                      L.is_split, L.is_relative, L.depends_on_lane, L.const_lo, L.const_hi, L.lower0, L.n_lower, L.upper0, L.n_upper);
        k.listing += line;
    }
    for (int i = 0; i < prog.n_bodies; ++i) {
        const TadpBody &B = prog.bodies[i];
        std::string t;
        for (int q = 0; q < TADP_BODY_STEPS && B.steps[q]; ++q) {
            char b2[40];
            if (B.steps[q] & 0x80) std::snprintf(b2, sizeof b2, " ld%d(load %d fetch %d op %d)", B.steps[q] & 3, B.load[B.steps[q] & 3], (B.steps[q] >> 4) & 7, (B.steps[q] >> 2) & 3);
            else std::snprintf(b2, sizeof b2, " s%d", B.steps[q]);
            t += b2;
        }
        std::snprintf(line, sizeof line, "; body %d loop_kind=%d term=%d inv=(%d:%d,%d:%d) steps:%s\n", i, B.loop_kind, B.term, B.inv_kind[0], B.inv_value[0],
                      B.inv_kind[1], B.inv_value[1], t.c_str());
        k.listing += line;
    }
    for (int i = 0; i < prog.n_rows; ++i) {
        std::snprintf(line, sizeof line, "; row %d (%d +%s ) / %d\n", i, prog.rows[i].c0, coefs(prog.rows[i].coef).c_str(), prog.rows[i].den);
        k.listing += line;
    }
}

}  // namespace

void emit_plain_kernel(Gen &g, Kernel &k, int root, const std::vector<std::vector<TadpRow>> &lower,
                       const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards, bool allow_split)
{
    count_uses(g, root);
    emit_kernel(g, k, root, lower, upper, guards, allow_split, false);
}

// workspace needs and launches of a kernel with its auxiliary kernels
static void account(tad_plan &p, Kernel &k)
{
    std::function<void(const Kernel &)> walk = [&](const Kernel &x) {
        if (x.ew.empty() && x.contract.empty() && x.prog.zsplit > 1)   // (line-sum kernels keep their shares in prog too)
            p.partial_bytes = std::max(p.partial_bytes, (size_t(x.prog.zsplit) + 1) * size_t(x.prog.part_limit) * 4);
        for (const TadcProgram &cp : x.contract)
            if (cp.ksplit > 1)
                p.partial_bytes = std::max(p.partial_bytes, size_t(cp.ksplit) * size_t(cp.M.extent) * size_t(cp.N.extent) * size_t(cp.Z.extent) * 4);
        for (const Kernel &y : x.pre) walk(y);
    };
    walk(k);
    p.aux_bytes = std::max(p.aux_bytes, k.aux_bytes);
    std::function<int(const Kernel &)> launches = [&](const Kernel &x) {
        int n = 0;
        if (!x.ew.empty()) n = 1;
        else if (x.contract.empty()) n = 1 + (x.prog.zsplit > 1 ? 1 + (x.prog.write_only_live && x.line.empty() ? 1 : 0) : 0);
        for (const TadcProgram &cp : x.contract) n += 1 + (cp.ksplit > 1 ? 1 : 0);
        for (const Kernel &y : x.pre) n += launches(y);
        return n;
    };
    k.stats.n_launches = launches(k);
}

// ---------------------------------------------------------------------------------------
// forward: outer variables are the output indices, every sum is a bound loop
// ---------------------------------------------------------------------------------------
namespace {

// kernels that run over the output box: outer variables are the output indices alpha
void setup_alpha_gen(tad_plan &p, Gen &g)
{
    g.n_outer = p.n_out; g.kappa = 0;
    const int nidx = p.n_out + p.n_sum;
    g.a_c0.assign(nidx, 0); g.a_coef.assign(nidx, std::vector<int64_t>(TADP_MAX_VARS, 0)); g.a_free_ok.assign(nidx, false);
    for (int d = 0; d < p.n_out; ++d) {
        g.new_var(0, p.out_shape[d]);
        g.a_coef[d][d] = 1; g.a_free_ok[d] = true;
    }
}

void finish_alpha_kernel(tad_plan &p, Gen &g, Kernel &k, int root)
{
    count_uses(g, root);
    g.lane_var = p.n_out - 1;
    TadpProgram &prog = k.prog;
    int64_t stride = 1;
    for (int d = p.n_out - 1; d >= 0; --d) {
        prog.outer_lo[d] = 0; prog.outer_ext[d] = to_i32(p.out_shape[d]);
        prog.out_coef[d] = to_i32(stride);
        stride *= p.out_shape[d];
    }
    prog.out_base = 0; prog.out_limit = to_i32(p.out_elems);
    prog.accumulate = 0; prog.write_only_live = 0;
    emit_kernel(g, k, root, {}, {}, {}, true);
    finish_stats(g, k, false, p.out_elems, 0, false);
    account(p, k);
}

}  // namespace

void generate_forward(tad_plan &p)
{
    Kernel &k = p.forward;
    std::memset(&k.prog, 0, sizeof k.prog);
    k.out_arg = -1; k.access = -1;
    Gen g(p, -1);
    setup_alpha_gen(p, g);
    int root = g.val((int)p.nodes.size() - 1, 0);
    finish_alpha_kernel(p, g, k, root);
}

// ---------------------------------------------------------------------------------------
// staging: the adjoint  df * d f / d s  of a top-level sum node s depends on alpha only and
// is shared by every gradient whose leaf sits inside that sum.  When it contains a sum of its
// own (so that re-evaluating it per term would repeat a whole inner loop) it is evaluated
// once per alpha by a kernel of its own into the workspace and read like df afterwards.
// ---------------------------------------------------------------------------------------
void generate_stages(tad_plan &p)
{
    const int root = (int)p.nodes.size() - 1;
    for (int n = 0; n < root; ++n) {
        const NodeH &nd = p.nodes[n];
        if (!nd.reachable || nd.op != TAD_OP_SUM || nd.scope != 0) continue;
        if (p.n_args + 1 + (int)p.stages.size() >= TADP_MAX_PTRS - (p.opt.saved_forward ? 1 : 0)) break;
        Gen g(p, -1);
        g.use_f = p.opt.saved_forward != 0;
        try {
            setup_alpha_gen(p, g);
            std::vector<int64_t> dfA(size_t(p.n_out) * g.n_idx(), 0), dfOff(p.n_out, 0);
            for (int d = 0; d < p.n_out; ++d) dfA[size_t(d) * g.n_idx() + d] = 1;
            int df_inst = g.make_load(p.n_args, dfA, dfOff, p.n_out, p.out_shape, 0, 0);
            int adj = g.differentiate(df_inst, n);
            if (adj < 0 || adj == df_inst) continue;
            count_uses(g, adj);
            bool has_sum = false;
            for (const Inst &in : g.inst) if (in.uses && in.op == I_SUM) has_sum = true;
            // with the forward output at hand the adjoint may be a few element-wise operations on df and f:
            // still evaluated once per alpha, so that the gradient loops read one tensor instead of two
            bool reads_f = false;
            for (const Inst &in : g.inst) if (in.uses && in.op == I_LOAD && g.loads[in.load].ptr == TADP_F_SLOT) reads_f = true;
            if (!has_sum && !reads_f) continue;
            Kernel k;
            std::memset(&k.prog, 0, sizeof k.prog);
            k.out_arg = -1; k.access = -1;
            finish_alpha_kernel(p, g, k, adj);
            p.stages.push_back(k);
            p.stage_node.push_back(n);
        } catch (const Unsupported &) {
            continue;      // too large to stage: the gradients recompute it
        }
    }
}

// ---------------------------------------------------------------------------------------
// backward of one index expression (Sec. 5.3: Delta, Omega, I/K/C, Omega', Sigma, accumulate)
// ---------------------------------------------------------------------------------------
void generate_backward(tad_plan &p, int q)
{
    AccessPlan &ap = p.access[q];
    p.backward.emplace_back();
    Kernel &k = p.backward.back();
    std::memset(&k.prog, 0, sizeof k.prog);
    k.out_arg = ap.arg; k.access = q;
    const int kidx = (int)p.backward.size() - 1;
    const bool first_of_arg = p.arg_kernels[ap.arg].empty();
    p.arg_kernels[ap.arg].push_back(kidx);
    const bool zero_fill = p.arg_zero_fill[ap.arg];

    Gen g(p, q);
    g.use_f = p.opt.saved_forward != 0;
    const int R = ap.R, kap = ap.kappa, n = ap.n, rank = ap.rank;
    // outer variables: beta itself when the map is onto the whole argument lattice, else x'
    const bool by_beta = !ap.masked;
    g.n_outer = by_beta ? rank : R;
    g.kappa = kap;
    const int nidx = p.n_out + p.n_sum;
    g.a_c0.assign(nidx, 0); g.a_coef.assign(nidx, std::vector<int64_t>(TADP_MAX_VARS, 0)); g.a_free_ok.assign(nidx, false);
    // the affine map alpha_hat = c0 + Mu u + K z
    Mat Mu(n, std::max(1, g.n_outer));
    std::vector<int64_t> c0(n, 0);
    std::vector<int64_t> ulo(g.n_outer), uhi(g.n_outer);
    if (by_beta) {
        // x' = U (beta - o)  =>  alpha_hat_0 = V_R U beta - V_R U o
        for (int d = 0; d < n; ++d)
            for (int c = 0; c < rank; ++c) {
                int64_t s = 0;
                for (int j = 0; j < R; ++j) s = add_ck(s, mul_ck(ap.V(d, j), ap.U(j, c)));
                Mu(d, c) = s;
                c0[d] = sub_ck(c0[d], mul_ck(s, ap.off[c]));
            }
        for (int c = 0; c < rank; ++c) { ulo[c] = 0; uhi[c] = p.arg_shape[ap.arg][c] - 1; }
    } else {
        for (int d = 0; d < n; ++d) for (int j = 0; j < R; ++j) Mu(d, j) = ap.V(d, j);
        for (int j = 0; j < R; ++j) { ulo[j] = ap.xlo[j]; uhi[j] = ap.xhi[j]; }
    }
    for (int j = 0; j < g.n_outer; ++j) g.new_var(0, uhi[j] - ulo[j] + 1);
    for (int col = 0; col < kap; ++col) g.new_var(1, kernel_col_extent(ap, col));
    for (int c = 0; c < n; ++c) {
        int d = ap.idx_pos[c];
        g.a_free_ok[d] = true;
        g.a_c0[d] = c0[c];
        for (int j = 0; j < g.n_outer; ++j) g.a_coef[d][j] = Mu(c, j);
        for (int col = 0; col < kap; ++col) g.a_coef[d][g.n_outer + col] = ap.V(c, R + col);
    }
    // df[alpha]: the sum indices are ignored when indexing df (Sec. 5.2)
    std::vector<int64_t> dfA(size_t(p.n_out) * nidx, 0), dfOff(p.n_out, 0);
    for (int d = 0; d < p.n_out; ++d) dfA[size_t(d) * nidx + d] = 1;
    int df_inst = g.make_load(p.n_args, dfA, dfOff, p.n_out, p.out_shape, ap.scope, ap.scope);
    for (size_t st = 0; st < p.stages.size(); ++st) g.staged[p.stage_node[st]] = p.n_args + 1 + (int)st;
    int root = g.differentiate(df_inst);
    if (root < 0) throw BadExpr("internal: index expression has no path to the root");
    for (int slot : g.stages_used) k.stages_used.push_back(slot - p.n_args - 1);
    count_uses(g, root);

    // Lane variable: a variable along which df is contiguous and which fills a warp, if there is
    // one; otherwise (and for the loop order always) the smallest estimated cost.
    const TadpLoad dfL = g.loads[g.inst[df_inst].load];
    int forced_lane = -1;
    for (int v = 0; v < g.n_outer + kap; ++v)
        if (std::abs(dfL.coef[v]) == 1 && g.vars[v].ext >= 32 &&
            (forced_lane < 0 || g.vars[v].ext > g.vars[forced_lane].ext ||
             (g.vars[v].ext == g.vars[forced_lane].ext && g.vars[v].kind == 1)))
            forced_lane = v;
    double best = -1; std::vector<int> best_order(kap); int best_lane = -1;
    auto search = [&](int forced_lane) {
    std::vector<int> perm(kap);
    for (int l = 0; l < kap; ++l) perm[l] = l;
    best = -1; best_order = perm; best_lane = -1;
    do {
        g.zorder = perm; g.zpos.assign(kap, 0);
        for (int l = 0; l < kap; ++l) g.zpos[perm[l]] = l;
        ap.zorder = perm;
        if (kap >= 2) compute_bounds(ap);
        for (int v = 0; v < g.n_outer + kap; ++v) {
            if (forced_lane >= 0 && v != forced_lane) continue;
            if (g.vars[v].ext < 2 && g.n_outer + kap > 1) continue;
            double c = schedule_cost(g, root, v);
            if (kap >= 2) {
                // A loop whose bounds differ from lane to lane pays for a range per element every time it is
                // entered: such a loop belongs outside the loops whose ranges the whole warp shares.
                double entries = 1;
                bool any_dep = false;
                for (int u = 0; u < g.n_outer; ++u) entries *= u == v ? std::ceil((double)g.vars[u].ext / 32.0) : (double)g.vars[u].ext;
                for (int l = 0; l < kap; ++l) {
                    bool dep = false;
                    auto reads_lane = [&](const BoundRowH &h) {
                        if (v >= g.n_outer) { for (int m = 0; m < l; ++m) if (perm[m] == v - g.n_outer && h.cz[m]) return true; return false; }
                        if (!by_beta) return h.cx[v] != 0;
                        int64_t sum = 0;
                        for (int j = 0; j < R; ++j) sum += h.cx[j] * ap.U(j, v);
                        return sum != 0;
                    };
                    for (const BoundRowH &h : ap.lower[l]) dep = dep || reads_lane(h);
                    for (const BoundRowH &h : ap.upper[l]) dep = dep || reads_lane(h);
                    // every entry of a loop costs its set-up, so the loop with the most trips belongs innermost
                    // (a loop over the lane variable makes one trip per 512 values at the widest shape)
                    c += entries * 50.0;
                    if (dep) { c += entries * 600.0; any_dep = true; }
                    const int lv = g.n_outer + perm[l];
                    entries *= lv == v ? std::ceil((double)g.vars[lv].ext / 512.0) : (double)g.vars[lv].ext;
                }
                // ... and everything inside it runs under per-element masks and start offsets, with the lanes
                // whose range is shorter idle: measured about three times the cost per term (cfg5 dx)
                if (any_dep) c *= 3.0;
            }
            c /= std::min(1.0, (double)g.vars[v].ext / 32.0);
            if (std::abs(dfL.coef[v]) == 1) c *= 0.999;
            if (g.vars[v].kind == 1) c *= 0.9999;
            if (best < 0 || c < best) { best = c; best_order = perm; best_lane = v; }
        }
    } while (std::next_permutation(perm.begin(), perm.end()));
    };
    search(forced_lane);
    if (forced_lane >= 0) {
        // ... unless another variable is estimated to be far cheaper (the strided loads of the forced
        // choice cost a transaction per lane: cfg2 da reads b[j, k] with one lane per j)
        const double forced_cost = best; const std::vector<int> forced_order = best_order; const int forced = best_lane;
        search(-1);
        if (!(best >= 0 && best * 2.5 < forced_cost)) { best = forced_cost; best_order = forced_order; best_lane = forced; }
    }
    if (best_lane < 0) best_lane = 0;
    g.zorder = best_order; g.zpos.assign(kap, 0);
    for (int l = 0; l < kap; ++l) g.zpos[best_order[l]] = l;
    g.lane_var = best_lane;
    ap.lane_var = best_lane;
    ap.zorder = best_order;
    compute_bounds(ap);

    // bound rows and guards over the kernel variables
    std::vector<int64_t> vlo(TADP_MAX_VARS, 0), vhi(TADP_MAX_VARS, 0);
    for (int j = 0; j < g.n_outer; ++j) { vlo[j] = ulo[j]; vhi[j] = uhi[j]; }
    for (int col = 0; col < kap; ++col) {
        // generous range of a kernel coordinate: z = (V^-1 alpha_hat)_{R+col} over the box, x' part aside
        int64_t mag = 0;
        for (int d = 0; d < n; ++d)
            mag = add_ck(mag, mul_ck(std::llabs(ap.Vinv(R + col, d)), std::max(std::llabs(ap.box_lo[d]), std::llabs(ap.box_hi[d]))));
        vlo[g.n_outer + col] = -mag; vhi[g.n_outer + col] = mag;
    }
    auto convert = [&](const BoundRowH &h, int loop) {
        TadpRow r{};
        r.den = to_i32(h.den);
        int64_t c = h.c0;
        std::vector<int64_t> cu(g.n_outer, 0);
        if (by_beta) {
            for (int col = 0; col < rank; ++col) {
                int64_t s = 0;
                for (int j = 0; j < R; ++j) s = add_ck(s, mul_ck(h.cx[j], ap.U(j, col)));
                cu[col] = s;
                c = sub_ck(c, mul_ck(s, ap.off[col]));
            }
        } else for (int j = 0; j < R; ++j) cu[j] = h.cx[j];
        r.c0 = to_i32(c);
        for (int j = 0; j < g.n_outer; ++j) r.coef[j] = to_i32(cu[j]);
        for (int m = 0; m < loop; ++m) r.coef[g.n_outer + ap.zorder[m]] = to_i32(h.cz[m]);
        check_row_range(r, vlo, vhi);
        return r;
    };
    std::vector<std::vector<TadpRow>> lower(kap), upper(kap);
    for (int l = 0; l < kap; ++l) {
        for (const BoundRowH &h : ap.lower[l]) lower[l].push_back(convert(h, l));
        for (const BoundRowH &h : ap.upper[l]) upper[l].push_back(convert(h, l));
    }
    std::vector<TadpRow> guards;
    for (const BoundRowH &h : ap.guards) {
        TadpRow r = convert(h, 0);
        // drop guards that hold on the whole outer box
        int64_t mx = r.c0;
        for (int j = 0; j < g.n_outer; ++j) mx += (int64_t)r.coef[j] * (r.coef[j] > 0 ? uhi[j] : ulo[j]);
        if (mx > 0) guards.push_back(r);
    }

    TadpProgram &prog = k.prog;
    for (int j = 0; j < g.n_outer; ++j) { prog.outer_lo[j] = to_i32(ulo[j]); prog.outer_ext[j] = to_i32(uhi[j] - ulo[j] + 1); }
    // output offset
    std::vector<int64_t> ostride(rank, 1);
    for (int r = rank - 2; r >= 0; --r) ostride[r] = ostride[r + 1] * p.arg_shape[ap.arg][r + 1];
    if (by_beta) {
        prog.out_base = 0;
        for (int r = 0; r < rank; ++r) prog.out_coef[r] = to_i32(ostride[r]);
    } else {
        // beta = o + U^-1[:, :R] diag(alpha) x'
        Mat Uinv = unimodular_inverse(ap.U);
        int64_t base = 0;
        for (int r = 0; r < rank; ++r) base = add_ck(base, mul_ck(ostride[r], ap.off[r]));
        prog.out_base = to_i32(base);
        for (int j = 0; j < R; ++j) {
            int64_t s = 0;
            for (int r = 0; r < rank; ++r) s = add_ck(s, mul_ck(ostride[r], mul_ck(Uinv(r, j), ap.inv[j])));
            prog.out_coef[j] = to_i32(s);
        }
    }
    prog.out_limit = to_i32(p.arg_elems[ap.arg]);
    prog.accumulate = (zero_fill || !first_of_arg) ? 1 : 0;
    prog.write_only_live = ap.masked ? 1 : 0;
    emit_kernel(g, k, root, lower, upper, guards, true);
    int64_t terms = 1;
    for (int d = 0; d < n; ++d) terms = mul_ck(terms, ap.box_hi[d] - ap.box_lo[d] + 1);
    finish_stats(g, k, true, p.arg_elems[ap.arg], terms, zero_fill && first_of_arg);
    account(p, k);
    if (zero_fill && first_of_arg) k.stats.n_launches += 1;
}

}  // namespace tad

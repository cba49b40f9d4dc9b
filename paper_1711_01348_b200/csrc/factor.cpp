// Expression optimisation pass (host only): the clean-up step that Sec. 6 names as missing.
//
// A kernel evaluates  out = sum over loops of a term.  When the term is a polynomial in index
// expressions, distributing its products turns it into monomials, and in each monomial the
// summation can be pushed inside: factors that do not read a summed variable leave the sum, a sum
// over a product of two factors is a contraction (run by the tile kernel), a sum over one factor
// is a contraction with a tensor of ones, and a sum whose whole index space is small is evaluated
// by a small interpreter kernel.  Intermediate results live in auxiliary tensors in the workspace;
// the kernels that fill them run before the kernel itself, which then reads them like arguments.
// Contractions that stream the same operand over the same summed variables are merged: their
// second operands become column blocks of one matrix, so the big operand crosses HBM once.
// The result is the same sum in another association; the statistics of the kernel (algorithmic
// bytes and flops) are taken from the expression as written, before this pass.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <functional>
#include <set>

#include "gen.h"

namespace tad {

namespace {

constexpr double SMALL_SPACE = double(1 << 24);     // index spaces up to this size are summed by an interpreter kernel
constexpr double MIN_SPACE = double(1 << 15);       // kernels with a smaller index space stay as they are
constexpr double MIN_GAIN = 6.0;                    // a contraction must shrink its index space at least this much
constexpr size_t MAX_MONOS = 16;
constexpr size_t MAX_DEGREE = 6;

struct Mono { double c = 1; std::vector<int> atoms; };
using Poly = std::vector<Mono>;

struct Tensor {                       // auxiliary tensor: dense, last variable fastest, plus a column index for merged ones
    std::vector<int> vars;            // parent variables that index it
    int64_t cols = 1;                 // merged tensors: number of columns (fastest index)
    int64_t elems = 0;
    std::vector<int64_t> stride;      // per entry of vars
};

struct Node {                         // a kernel that fills (part of) a tensor
    int kind = 0;                     // 0: interpreter, 1: contraction
    int tensor = -1;
    int64_t col0 = 0;                 // interpreter nodes writing a column block of a merged tensor
    std::vector<int> dims, sums;      // interpreter: output variables (beside the block's own), summed variables
    Poly poly;                        // interpreter: the summand
    int group = -1;                   // contraction: which group
    int table_inst = -1, table_load = -1;   // kind 2: a function of one index expression, evaluated over that argument's elements
};

struct Request { std::vector<int> b_atoms; uint32_t nmask = 0; int load_id = -1; int64_t col0 = 0, width = 1; };
struct Group {
    int a_inst = -1; uint32_t kmask = 0;
    std::vector<Request> reqs;
    int t_tensor = -1, x_tensor = -1;
    int64_t cols = 0;                 // merged: columns in use (the tensors' rows are padded to whole 16-byte pieces)
    bool u_trick = false;             // single request on ones with the output indexed by the operand's own row
    int64_t u_g = 1, u0 = 0, u_ext = 0;
};

struct Factorizer {
    Gen &w;
    Kernel &k;
    const int nv0;                                    // parent variables known at the start (more are found in sums)
    std::vector<int64_t> vlo, vext;
    std::vector<bool> can_sum;                        // summed variable with a fixed range
    std::vector<Tensor> tensors;
    std::vector<Node> nodes;
    std::vector<Group> groups;
    std::map<int, int> load_tensor;                   // load id -> tensor (auxiliary loads)
    std::map<int, int> memo;
    bool changed = false;
    bool allow_sums = true;                           // false: only function tables (kernels with guards)
    int n_outer_vars = 0;
    bool has_loops = false;                           // the kernel has summation loops around its term
    std::map<int, int> table_memo;                    // instance -> load of its table

    Factorizer(Gen &gen, Kernel &kern) : w(gen), k(kern), nv0((int)gen.vars.size()), vlo(TADP_MAX_VARS, 0), vext(TADP_MAX_VARS, 1), can_sum(TADP_MAX_VARS, false) {}

    double space(uint32_t mask) const
    {
        double s = 1;
        for (int v = 0; v < TADP_MAX_VARS; ++v) if (mask & (1u << v)) s *= (double)std::max<int64_t>(1, vext[v]);
        return s;
    }
    uint32_t deps_of(const std::vector<int> &atoms) const { uint32_t d = 0; for (int a : atoms) d |= w.inst[a].deps; return d; }

    // ---- polynomial expansion -----------------------------------------------------------------
    static void add_mono(Poly &p, Mono m)
    {
        std::sort(m.atoms.begin(), m.atoms.end());
        for (Mono &o : p) if (o.atoms == m.atoms) { o.c += m.c; return; }
        p.push_back(std::move(m));
    }
    static bool product(const Poly &a, const Poly &b, Poly &out)
    {
        out.clear();
        for (const Mono &x : a)
            for (const Mono &y : b) {
                Mono m; m.c = x.c * y.c; m.atoms = x.atoms; m.atoms.insert(m.atoms.end(), y.atoms.begin(), y.atoms.end());
                if (m.atoms.size() > MAX_DEGREE) return false;
                add_mono(out, std::move(m));
                if (out.size() > MAX_MONOS) return false;
            }
        return true;
    }
    bool expand(int i, Poly &out)
    {
        const Inst in = w.inst[i];
        auto atom = [&]() { out.clear(); Mono m; m.atoms = {i}; out.push_back(m); return true; };
        Poly a, b;
        switch (in.op) {
        case I_CONST: { out.clear(); Mono m; m.c = in.imm; out.push_back(m); return true; }
        case I_NEG: if (!expand(in.a, out)) return atom(); for (Mono &m : out) m.c = -m.c; return true;
        case I_MULC: if (!expand(in.a, out)) return atom(); for (Mono &m : out) m.c *= in.imm; return true;
        case I_ADDC: { if (!expand(in.a, out)) return atom(); Mono m; m.c = in.imm; add_mono(out, m); return out.size() <= MAX_MONOS || atom(); }
        case I_ADD: case I_SUB:
            if (!expand(in.a, a) || !expand(in.b, b)) return atom();
            out = a;
            for (Mono &m : b) { if (in.op == I_SUB) m.c = -m.c; add_mono(out, m); }
            return out.size() <= MAX_MONOS || atom();
        case I_MUL:
            if (!expand(in.a, a) || !expand(in.b, b) || !product(a, b, out)) return atom();
            return true;
        case I_SQR:
            if (!expand(in.a, a) || !product(a, a, out)) return atom();
            return true;
        case I_POWI: {
            if (in.ipow < 2 || in.ipow > 4 || !expand(in.a, a) || a.size() > 1) return atom();
            out = a;
            for (int n = 1; n < in.ipow; ++n) { Poly t; if (!product(out, a, t)) return atom(); out = t; }
            return true;
        }
        default: return atom();
        }
    }

    // ---- instance construction ----------------------------------------------------------------
    int build_mono(const Mono &m, const std::vector<int> &atoms)
    {
        int r = -1;
        for (int a : atoms) r = r < 0 ? a : w.bin(I_MUL, r, a);
        if (r < 0) return w.konst((float)m.c);
        return w.mulc(r, (float)m.c);
    }
    int build_poly(const Poly &p)
    {
        int r = -1;
        for (const Mono &m : p) { const int t = build_mono(m, m.atoms); r = r < 0 ? t : w.bin(I_ADD, r, t); }
        return r < 0 ? w.konst(0.f) : r;
    }
    int wrap_sums(int body, const std::vector<int> &vars)
    {
        // innermost first in `vars`; the same variables as the sums this replaces
        for (int v : vars) {
            Inst s; s.op = I_SUM; s.a = body; s.var = v; s.lo = vlo[v]; s.hi = vlo[v] + vext[v] - 1;
            s.deps = w.inst[body].deps & ~(1u << v);
            s.adeps = w.inst[body].adeps & ~(1u << (16 + v));
            body = w.intern(s);
            w.vars[v].sum_inst = body;
        }
        return body;
    }

    // ---- auxiliary tensors ---------------------------------------------------------------------
    int new_tensor(const std::vector<int> &vars, int64_t cols)
    {
        Tensor t; t.vars = vars; t.cols = cols;
        t.stride.assign(vars.size(), 0);
        int64_t s = cols;
        for (int d = (int)vars.size() - 1; d >= 0; --d) { t.stride[d] = s; s = mul_ck(s, std::max<int64_t>(1, vext[vars[d]])); }
        t.elems = s;
        if (t.elems >= (int64_t(1) << 31)) throw Overflow();
        tensors.push_back(t);
        return (int)tensors.size() - 1;
    }
    // load of tensor t at its own variables (plus a fixed column and optional column variables)
    int tensor_load(int t, int64_t col0, const std::vector<std::pair<int, int64_t>> &col_vars = {})
    {
        const Tensor &T = tensors[t];
        TadpLoad L{};
        L.ptr = -1 - t;                      // patched to the pointer slot when the kernels are built
        int64_t base = col0;
        for (size_t d = 0; d < T.vars.size(); ++d) {
            L.coef[T.vars[d]] = to_i32(T.stride[d]);
            base = sub_ck(base, mul_ck(T.stride[d], vlo[T.vars[d]]));
        }
        for (auto &cv : col_vars) { L.coef[cv.first] = to_i32(add_ck(L.coef[cv.first], cv.second)); base = sub_ck(base, mul_ck(cv.second, vlo[cv.first])); }
        L.base = to_i32(base);
        L.limit = to_i32(T.elems);
        if ((int)w.loads.size() >= 64) throw Unsupported("too many loads");
        w.loads.push_back(L);
        const int id = (int)w.loads.size() - 1;
        load_tensor[id] = t;
        Inst in; in.op = I_LOAD; in.load = id;
        for (int v = 0; v < TADP_MAX_VARS; ++v) if (L.coef[v]) in.deps |= 1u << v;
        return w.intern(in);
    }
    std::vector<int> vars_of(uint32_t mask) const { std::vector<int> r; for (int v = 0; v < TADP_MAX_VARS; ++v) if (mask & (1u << v)) r.push_back(v); return r; }

    // T[dims] = sum over `sums` of poly, by an interpreter kernel
    int small_sum(uint32_t dims, uint32_t sums, const Poly &poly)
    {
        const int t = new_tensor(vars_of(dims), 1);
        Node n; n.kind = 0; n.tensor = t; n.dims = vars_of(dims); n.sums = vars_of(sums); n.poly = poly;
        nodes.push_back(n);
        changed = true;
        return tensor_load(t, 0);
    }

    // sum over kmask of  a_inst * product(b_atoms): a request in the group of (a_inst, kmask)
    int request(int a_inst, uint32_t kmask, const std::vector<int> &b_atoms)
    {
        int gi = -1;
        for (size_t i = 0; i < groups.size(); ++i) if (groups[i].a_inst == a_inst && groups[i].kmask == kmask) gi = (int)i;
        if (gi < 0) { Group G; G.a_inst = a_inst; G.kmask = kmask; groups.push_back(G); gi = (int)groups.size() - 1; }
        Group &G = groups[gi];
        Request r; r.b_atoms = b_atoms; std::sort(r.b_atoms.begin(), r.b_atoms.end());
        r.nmask = deps_of(b_atoms) & ~kmask;
        for (const Request &o : G.reqs) if (o.b_atoms == r.b_atoms) { Inst in; in.op = I_LOAD; in.load = o.load_id; return w.intern(in); }
        // placeholder load: offsets are set when the group's layout is known
        TadpLoad L{}; L.ptr = -1000 - gi;
        const uint32_t out_mask = (w.inst[a_inst].deps & ~kmask) | r.nmask;
        for (int v = 0; v < TADP_MAX_VARS; ++v) if (out_mask & (1u << v)) L.coef[v] = 1;     // marks the dependence only
        w.loads.push_back(L);
        r.load_id = (int)w.loads.size() - 1;
        G.reqs.push_back(r);
        Inst in; in.op = I_LOAD; in.load = r.load_id; in.deps = out_mask;
        changed = true;
        return w.intern(in);
    }

    bool is_plain_load(int i) const { return w.inst[i].op == I_LOAD; }

    // ---- summation of one monomial over the variables of `emask` --------------------------------
    // returns the instance of  sum_emask (c * product(atoms)), or -1 when nothing is gained
    int sum_mono(const Mono &m, uint32_t emask)
    {
        std::vector<int> pre, red;
        for (int a : m.atoms) ((w.inst[a].deps & emask) ? red : pre).push_back(a);
        double mult = 1;
        uint32_t live = emask & deps_of(red);
        for (int v = 0; v < TADP_MAX_VARS; ++v) if ((emask & (1u << v)) && !(live & (1u << v))) mult *= (double)vext[v];
        while (live) {
            const uint32_t d_all = deps_of(red);
            if (space(d_all) <= SMALL_SPACE) {
                // everything that is left is small: one interpreter kernel; factors over its output variables join it
                const uint32_t d_out = d_all & ~live;
                Mono body; body.atoms = red;
                std::vector<int> keep;
                for (int a : pre) { if ((w.inst[a].deps & ~d_out) == 0 && w.inst[a].deps) body.atoms.push_back(a); else keep.push_back(a); }
                pre = keep;
                red = {small_sum(d_out, live, Poly{body})};
                live = 0;
                break;
            }
            // the variable whose factors span the smallest index space
            int best = -1; double best_cost = 0, best_out = 0; uint32_t best_k = 0; std::vector<int> best_s;
            for (int v = 0; v < TADP_MAX_VARS; ++v) {
                if (!(live & (1u << v))) continue;
                std::vector<int> sv;
                for (int a : red) if (w.inst[a].deps & (1u << v)) sv.push_back(a);
                uint32_t kv = 0;
                for (int u = 0; u < TADP_MAX_VARS; ++u) {
                    if (!(live & (1u << u))) continue;
                    bool only = true;
                    for (int a : red) if ((w.inst[a].deps & (1u << u)) && std::find(sv.begin(), sv.end(), a) == sv.end()) only = false;
                    if (only) kv |= 1u << u;
                }
                const double cost = space(deps_of(sv)), outsp = space(deps_of(sv) & ~kv);
                if (best < 0 || cost < best_cost || (cost == best_cost && outsp < best_out)) { best = v; best_cost = cost; best_out = outsp; best_k = kv; best_s = sv; }
            }
            if (best < 0 || best_cost / best_out < MIN_GAIN) return -1;
            int t_inst = -1;
            if (best_cost <= SMALL_SPACE) {
                Mono body; body.atoms = best_s;
                t_inst = small_sum(deps_of(best_s) & ~best_k, best_k, Poly{body});
            } else {
                // contraction: the factor with the largest index space is streamed as it is, the others form the second operand
                int big = -1;
                for (int a : best_s) if (is_plain_load(a) && (big < 0 || space(w.inst[a].deps) > space(w.inst[big].deps))) big = a;
                if (big < 0) return -1;
                std::vector<int> rest;
                bool taken = false;
                for (int a : best_s) { if (a == big && !taken) { taken = true; continue; } rest.push_back(a); }
                if (!rest.empty() && space(deps_of(rest)) > SMALL_SPACE && !(rest.size() == 1 && is_plain_load(rest[0]))) return -1;
                // the streamed operand must bring enough rows of its own to fill tiles (variables that the second
                // operand reads too only number independent contractions)
                if (space(w.inst[big].deps & ~best_k & ~deps_of(rest)) < 64) return -1;
                // every summed variable must be read by the streamed operand or the second one
                t_inst = request(big, best_k, rest);
            }
            // the factors of best_s (one occurrence each) are replaced by the result
            std::vector<int> next;
            { std::vector<int> pool = best_s; for (int a : red) { auto it = std::find(pool.begin(), pool.end(), a); if (it != pool.end()) pool.erase(it); else next.push_back(a); } }
            next.push_back(t_inst);
            red = next;
            live &= ~best_k;
            // factors that no longer read a summed variable leave the sum
            std::vector<int> still;
            for (int a : red) ((w.inst[a].deps & live) ? still : pre).push_back(a);
            red = still;
        }
        std::vector<int> all = pre; all.insert(all.end(), red.begin(), red.end());
        Mono r; r.c = m.c * mult;
        return build_mono(r, all);
    }

    // sum over `vars` (innermost first) of the instance `body`
    int solve(const std::vector<int> &vars, int body)
    {
        uint32_t emask = 0;
        for (int v : vars) { if (!can_sum[v]) return -1; emask |= 1u << v; }
        Poly P;
        if (!expand(body, P) || P.empty()) return -1;
        if (space(w.inst[body].deps | emask) < MIN_SPACE) return -1;
        // monomials whose whole index space is small are summed together by one interpreter kernel per output set
        std::map<uint32_t, Poly> small;
        Poly rest;
        for (const Mono &m : P) {
            const uint32_t d = deps_of(m.atoms);
            if (space(d | emask) <= SMALL_SPACE && (d & emask)) small[d & ~emask].push_back(m);
            else rest.push_back(m);
        }
        // nothing but small monomials: the sum is cheap as it is
        if (rest.empty()) return -1;
        const size_t n_nodes = nodes.size(), n_tensors = tensors.size(), n_groups = groups.size();
        std::vector<size_t> n_reqs; for (const Group &G : groups) n_reqs.push_back(G.reqs.size());
        const bool was_changed = changed;
        int total = -1;
        bool ok = true;
        for (const Mono &m : rest) {
            const int t = sum_mono(m, emask);
            if (t < 0) { ok = false; break; }
            total = total < 0 ? t : w.bin(I_ADD, total, t);
        }
        if (!ok) {
            // leave the whole sum as it was
            nodes.resize(n_nodes); tensors.resize(n_tensors); groups.resize(n_groups);
            for (size_t i = 0; i < groups.size(); ++i) groups[i].reqs.resize(n_reqs[i]);
            changed = was_changed;
            return -1;
        }
        for (auto &kv : small) {
            double mult = 1;
            const uint32_t inner = emask & deps_of_poly(kv.second);
            for (int v = 0; v < TADP_MAX_VARS; ++v) if ((emask & (1u << v)) && !(inner & (1u << v))) mult *= (double)vext[v];
            int t = small_sum(kv.first, inner, kv.second);
            t = w.mulc(t, (float)mult);
            total = total < 0 ? t : w.bin(I_ADD, total, t);
        }
        return total;
    }
    uint32_t deps_of_poly(const Poly &p) const { uint32_t d = 0; for (const Mono &m : p) d |= deps_of(m.atoms); return d; }

    // ---- function tables ------------------------------------------------------------------------
    // An expression whose only leaf is one index expression of an argument (exp x[i + j], 1 - tanh^2 x[2i + 3j],
    // sin x[...]) takes as many distinct values as the argument has elements.  When the kernel would evaluate it
    // far more often than that, it is evaluated once per element of the argument into an auxiliary tensor of
    // the argument's shape, and the kernel reads that tensor through the same index expression.
    // returns the load id if instance i is such an expression (no sums, one load), else -1; cost: its operations
    int single_load(int i, double &cost, bool &transcendental)
    {
        const Inst &in = w.inst[i];
        switch (in.op) {
        case I_CONST: return -2;
        case I_LOAD: return w.loads[in.load].ptr >= 0 ? in.load : -1;
        case I_SUM: return -1;
        default: break;
        }
        if (in.op == I_EXP || in.op == I_LOG || in.op == I_SIN || in.op == I_COS || in.op == I_TANH || in.op == I_SINH || in.op == I_COSH ||
            in.op == I_DIV || (in.op == I_POWI && (in.ipow < 0 || in.ipow > 4))) { transcendental = true; cost += 8; }
        else cost += 1;
        const int a = single_load(in.a, cost, transcendental);
        if (a == -1) return -1;
        if (in.b < 0) return a;
        const int b = single_load(in.b, cost, transcendental);
        if (b == -1) return -1;
        if (a == -2) return b;
        if (b == -2) return a;
        return a == b ? a : -1;
    }
    int try_table(int i)
    {
        auto it = table_memo.find(i);
        if (it != table_memo.end()) return it->second;
        double cost = 0; bool tr = false;
        const int ld = single_load(i, cost, tr);
        if (ld < 0 || !tr) return -1;
        const TadpLoad L = w.loads[ld];
        // how often the kernel evaluates it: once per binding of its variables, and a value inside a loop is
        // evaluated again for every output that runs the loop
        uint32_t reach = w.inst[i].deps;
        if (reach >> n_outer_vars) reach |= (1u << n_outer_vars) - 1u;
        // a kernel with summation loops also tabulates the factors outside its sums when the table is not much
        // larger than the number of outputs: its terms are then products of index expressions (line sums)
        const double worth = (has_loops && !(w.inst[i].deps >> n_outer_vars)) ? 0.5 : 8.0;
        if (L.limit <= 0 || (double)L.limit * worth > space(reach) || L.limit > (1 << 26)) return -1;
        Tensor T; T.cols = 1; T.elems = L.limit;
        tensors.push_back(T);
        const int t = (int)tensors.size() - 1;
        Node n; n.kind = 2; n.tensor = t; n.table_inst = i; n.table_load = ld;
        nodes.push_back(n);
        TadpLoad N = L;
        N.ptr = -1 - t;
        w.loads.push_back(N);
        const int id = (int)w.loads.size() - 1;
        load_tensor[id] = t;
        Inst li; li.op = I_LOAD; li.load = id; li.deps = w.inst[i].deps; li.adeps = w.inst[i].adeps;
        const int r = w.intern(li);
        table_memo[i] = r;
        changed = true;
        return r;
    }

    // rewrites the sums below instance i; returns the (possibly new) instance
    int rewrite(int i)
    {
        auto it = memo.find(i);
        if (it != memo.end()) return it->second;
        const Inst in = w.inst[i];
        int r = i;
        if (in.op != I_CONST && in.op != I_LOAD && in.op != I_SUM) {
            const int tbl = try_table(i);
            if (tbl >= 0) { memo[i] = tbl; return tbl; }
        }
        if (in.op == I_SUM) {
            std::vector<int> vars{in.var};
            int body = in.a;
            while (w.inst[body].op == I_SUM) { vars.push_back(w.inst[body].var); body = w.inst[body].a; }
            std::reverse(vars.begin(), vars.end());            // innermost first
            // ranges of these variables
            int cur = i;
            while (w.inst[cur].op == I_SUM) {
                const Inst &s = w.inst[cur];
                vlo[s.var] = s.lo; vext[s.var] = std::max<int64_t>(0, s.hi - s.lo + 1); can_sum[s.var] = vext[s.var] > 0;
                cur = s.a;
            }
            const int nb = rewrite(body);
            const int solved = allow_sums ? solve(vars, nb) : -1;
            if (solved >= 0) r = solved;
            else if (nb != body) r = wrap_sums(nb, vars);
        } else if (in.op != I_CONST && in.op != I_LOAD) {
            const int a = rewrite(in.a), b = in.b >= 0 ? rewrite(in.b) : -1;
            if (a != in.a || b != in.b) {
                switch (in.op) {
                case I_NEG: r = w.neg(a); break;
                case I_MULC: r = w.mulc(a, in.imm); break;
                case I_ADDC: r = w.addc(a, in.imm); break;
                case I_POWI: r = w.powi(a, in.ipow); break;
                case I_ADD: case I_SUB: case I_MUL: case I_DIV: r = w.bin(in.op, a, b); break;
                default: r = w.un(in.op, a); break;
                }
            }
        }
        memo[i] = r;
        return r;
    }
};

// ---- translation of instances into a fresh generator with its own variable numbering -------------
struct Translator {
    Gen &src, &dst;
    std::vector<int> var_map;
    const std::vector<int> &slot_of_tensor;      // auxiliary tensor -> pointer slot
    std::map<int, int> memo;
    int flat_load = -1;                          // this load is read at element index = variable 0 (function tables)
    Translator(Gen &s, Gen &d, const std::vector<int> &slots) : src(s), dst(d), var_map(TADP_MAX_VARS, -1), slot_of_tensor(slots) {}
    int run(int i)
    {
        auto it = memo.find(i);
        if (it != memo.end()) return it->second;
        const Inst in = src.inst[i];
        int r = -1;
        switch (in.op) {
        case I_CONST: r = dst.konst(in.imm); break;
        case I_LOAD: {
            const TadpLoad &L = src.loads[in.load];
            TadpLoad N{};
            N.ptr = L.ptr < 0 ? slot_of_tensor[-1 - L.ptr] : L.ptr;
            N.base = L.base; N.limit = L.limit;
            uint32_t deps = 0;
            if (in.load == flat_load) { N.base = 0; N.coef[0] = 1; deps = 1u; }
            else for (int v = 0; v < TADP_MAX_VARS; ++v) {
                if (!L.coef[v]) continue;
                if (var_map[v] < 0) throw BadExpr("internal: variable outside the kernel");
                N.coef[var_map[v]] += L.coef[v];
                deps |= 1u << var_map[v];
            }
            int id = -1;
            for (size_t j = 0; j < dst.loads.size(); ++j) if (!std::memcmp(&dst.loads[j], &N, sizeof N)) id = (int)j;
            if (id < 0) {
                if ((int)dst.loads.size() >= TADP_MAX_LOADS) throw Unsupported("too many distinct loads in one kernel");
                dst.loads.push_back(N); id = (int)dst.loads.size() - 1;
            }
            Inst n; n.op = I_LOAD; n.load = id; n.deps = deps;
            r = dst.intern(n);
            break;
        }
        case I_SUM: {
            const int v = dst.new_var(2, std::max<int64_t>(0, in.hi - in.lo + 1));
            var_map[in.var] = v;
            const int body = run(in.a);
            Inst s; s.op = I_SUM; s.a = body; s.var = v; s.lo = in.lo; s.hi = in.hi;
            s.deps = dst.inst[body].deps & ~(1u << v);
            r = dst.intern(s);
            dst.vars[v].sum_inst = r;
            break;
        }
        case I_NEG: r = dst.neg(run(in.a)); break;
        case I_MULC: r = dst.mulc(run(in.a), in.imm); break;
        case I_ADDC: r = dst.addc(run(in.a), in.imm); break;
        case I_POWI: r = dst.powi(run(in.a), in.ipow); break;
        case I_ADD: case I_SUB: case I_MUL: case I_DIV: { const int a = run(in.a), b = run(in.b); r = dst.bin(in.op, a, b); break; }
        default: r = dst.un(in.op, run(in.a)); break;
        }
        memo[i] = r;
        return r;
    }
};

}  // namespace

static bool factor_kernel(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
                          const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards)
{
    tad_plan &p = g.p;
    // kernels with guards own elements without any term; the auxiliary kernels would evaluate index expressions there
    if (p.opt.debug_bounds || root < 0) return false;
    Gen w = g;                                    // the pass works on a copy: the caller's instances keep their meaning
    Factorizer F(w, k);
    F.allow_sums = guards.empty();
    F.n_outer_vars = g.n_outer;
    F.has_loops = g.kappa >= 1;
    const TadpProgram &prog = k.prog;
    for (int v = 0; v < g.n_outer; ++v) { F.vlo[v] = prog.outer_lo[v]; F.vext[v] = prog.outer_ext[v]; }
    // kernel-coordinate loops with fixed ranges that no other loop's bounds read can be summed away
    auto constant = [](const TadpRow &r) { for (int v = 0; v < TADP_MAX_VARS; ++v) if (r.coef[v]) return false; return true; };
    std::vector<int> zvars;
    for (int l = 0; l < g.kappa; ++l) {
        const int z = g.n_outer + g.zorder[l];
        zvars.push_back(z);
        bool fixed = !lower[l].empty() && !upper[l].empty();
        for (const TadpRow &r : lower[l]) fixed = fixed && constant(r);
        for (const TadpRow &r : upper[l]) fixed = fixed && constant(r);
        if (!fixed) {
            // bounding box of a loop whose bounds move with other variables: z >= every lower row, so z >= the largest
            // of their minima over the box of the variables they read (outer loops come first); the same from above
            if (lower[l].empty() || upper[l].empty()) return false;
            auto extreme = [&](const TadpRow &r, bool want_max) {
                int64_t num = r.c0;
                for (int v = 0; v < TADP_MAX_VARS; ++v) {
                    if (!r.coef[v]) continue;
                    const int64_t a = F.vlo[v], b = F.vlo[v] + std::max<int64_t>(1, F.vext[v]) - 1;
                    num += (int64_t)r.coef[v] * (((r.coef[v] > 0) == want_max) ? b : a);
                }
                return num;
            };
            int64_t lo = INT64_MIN, hi = INT64_MAX;
            for (const TadpRow &r : lower[l]) lo = std::max(lo, ceil_div(extreme(r, false), r.den));
            for (const TadpRow &r : upper[l]) hi = std::min(hi, floor_div(extreme(r, true), r.den));
            F.vlo[z] = lo; F.vext[z] = std::max<int64_t>(1, hi - lo + 1);
        }
        if (fixed) {
            int64_t lo = INT64_MIN, hi = INT64_MAX;
            for (const TadpRow &r : lower[l]) lo = std::max(lo, ceil_div(r.c0, r.den));
            for (const TadpRow &r : upper[l]) hi = std::min(hi, floor_div(r.c0, r.den));
            F.vlo[z] = lo; F.vext[z] = std::max<int64_t>(0, hi - lo + 1);
            F.can_sum[z] = F.vext[z] > 0;
        }
    }
    for (int l = 0; l < g.kappa; ++l)
        for (const std::vector<TadpRow> *rows : {&lower[l], &upper[l]})
            for (const TadpRow &r : *rows)
                for (int z : zvars) if (r.coef[z]) F.can_sum[z] = false;
    // ---- the sums inside the term, then the loops around it ----
    int term = F.rewrite(root);
    std::vector<int> summed;                      // kernel coordinates that the rewritten term no longer needs a loop for
    {
        std::vector<int> cand;
        for (int l = g.kappa - 1; l >= 0; --l) if (F.can_sum[zvars[l]]) cand.push_back(zvars[l]);
        if (!cand.empty() && F.allow_sums) {
            const int solved = F.solve(cand, term);
            if (solved >= 0) { term = solved; summed = cand; }
        }
    }
    int scale_r = scale >= 0 ? F.rewrite(scale) : -1;
    if (!F.changed) return false;
    if (scale_r >= 0) term = w.bin(I_MUL, term, scale_r);

    // ---- fusion: an element-wise kernel around one contraction becomes that contraction's epilogue -------------
    // What is left may be  h(S)  with h a chain of unary steps (and products with tensors laid out like the output)
    // and S a sum of monomials of which one holds the result T of a contraction sum_k A[m, k] B[n, k] and all others
    // are products of a factor over the row variables and a factor over the column variables.  Then S itself is a
    // contraction: the factors of T's monomial scale A and B, every other monomial adds one summation index
    // (A' = its row factor, B' = its column factor).  A' and B' are small pre-evaluated matrices, the finished sums
    // go through h in registers, and T never exists in memory.
    struct Fusion {
        bool on = false;
        int a_tensor = -1, b_tensor = -1;
        uint32_t mmask = 0, nmask = 0;
        int64_t cols = 0;
        std::vector<int> op; std::vector<float> imm; std::vector<int> load;    // epilogue steps, innermost first
    } fusion;
    if (summed.size() == (size_t)g.kappa) {
        std::vector<int> op; std::vector<float> imm; std::vector<int> lds;
        int cur = term;
        auto elementwise = [&](int i) {
            if (w.inst[i].op != I_LOAD) return false;
            const TadpLoad &L = w.loads[w.inst[i].load];
            for (int v = 0; v < TADP_MAX_VARS; ++v) if (L.coef[v] != (v < g.n_outer ? prog.out_coef[v] : 0)) return false;
            return L.ptr >= 0;
        };
        for (bool go = true; go && (int)op.size() < TADC_MAX_EPI;) {
            const Inst in = w.inst[cur];
            switch (in.op) {
            case I_NEG: op.push_back(TE_NEG); imm.push_back(0); lds.push_back(-1); cur = in.a; break;
            case I_EXP: op.push_back(TE_EXP); imm.push_back(0); lds.push_back(-1); cur = in.a; break;
            case I_TANH: op.push_back(TE_TANH); imm.push_back(0); lds.push_back(-1); cur = in.a; break;
            case I_SQR: op.push_back(TE_SQR); imm.push_back(0); lds.push_back(-1); cur = in.a; break;
            case I_MULC: op.push_back(TE_MULC); imm.push_back(in.imm); lds.push_back(-1); cur = in.a; break;
            case I_ADDC: op.push_back(TE_ADDC); imm.push_back(in.imm); lds.push_back(-1); cur = in.a; break;
            case I_MUL:
                if (elementwise(in.a) && !elementwise(in.b)) { op.push_back(TE_MUL_LOAD); imm.push_back(0); lds.push_back(w.inst[in.a].load); cur = in.b; }
                else if (elementwise(in.b) && !elementwise(in.a)) { op.push_back(TE_MUL_LOAD); imm.push_back(0); lds.push_back(w.inst[in.b].load); cur = in.a; }
                else go = false;
                break;
            default: go = false; break;
            }
        }
        Poly S;
        int t_group = -1, t_mono = -1, t_atom = -1, n_results = 0;
        if (F.expand(cur, S) && S.size() >= 1 && S.size() <= 6) {
            for (size_t mi = 0; mi < S.size(); ++mi)
                for (int a : S[mi].atoms) {
                    if (w.inst[a].op != I_LOAD) continue;
                    const int ptr = w.loads[w.inst[a].load].ptr;
                    if (ptr <= -1000) { ++n_results; t_group = -1000 - ptr; t_mono = (int)mi; t_atom = a; }
                }
        }
        uint32_t outer_mask = 0;
        for (int v = 0; v < g.n_outer; ++v) if (F.vext[v] > 1) outer_mask |= 1u << v;
        bool ok = n_results == 1 && t_group >= 0;
        if (ok) {
            const Group &G = F.groups[t_group];
            ok = G.reqs.size() == 1 && G.reqs[0].b_atoms.size() == 1 && F.is_plain_load(G.reqs[0].b_atoms[0]);
            if (ok) {
                fusion.mmask = w.inst[G.a_inst].deps & ~G.kmask;
                fusion.nmask = w.inst[G.reqs[0].b_atoms[0]].deps & ~G.kmask;
                ok = fusion.mmask && fusion.nmask && !(fusion.mmask & fusion.nmask) && ((fusion.mmask | fusion.nmask) & outer_mask) == outer_mask &&
                     !((fusion.mmask | fusion.nmask) & ~outer_mask & ~0u) ;
                // every other factor lives on the row side or on the column side
                for (const Mono &m : S)
                    for (int a : m.atoms) {
                        if (a == t_atom) continue;
                        const uint32_t d = w.inst[a].deps;
                        if ((d & ~fusion.mmask) && (d & ~fusion.nmask)) ok = false;
                    }
            }
        }
        if (ok) {
            Group &G = F.groups[t_group];
            int64_t kext = 1;
            for (int v = 0; v < TADP_MAX_VARS; ++v) if (G.kmask & (1u << v)) kext = mul_ck(kext, F.vext[v]);
            fusion.cols = kext + (int64_t)S.size() - 1;
            fusion.a_tensor = F.new_tensor(F.vars_of(fusion.mmask), fusion.cols);
            fusion.b_tensor = F.new_tensor(F.vars_of(fusion.nmask), fusion.cols);
            int64_t col = kext;
            for (size_t mi = 0; mi < S.size(); ++mi) {
                Mono ma, mb; ma.c = S[mi].c; mb.c = 1;
                bool t_seen = false;
                for (int a : S[mi].atoms) {
                    if (a == t_atom && !t_seen) { t_seen = true; continue; }
                    ((w.inst[a].deps & ~fusion.mmask) ? mb : ma).atoms.push_back(a);
                }
                Node na, nb;
                na.kind = nb.kind = 0; na.tensor = fusion.a_tensor; nb.tensor = fusion.b_tensor;
                if ((int)mi == t_mono) {
                    ma.atoms.push_back(G.a_inst); mb.atoms.push_back(G.reqs[0].b_atoms[0]);
                    na.col0 = nb.col0 = 0;
                    na.dims = F.vars_of(fusion.mmask | G.kmask); nb.dims = F.vars_of(fusion.nmask | G.kmask);
                } else {
                    na.col0 = nb.col0 = col++;
                    na.dims = F.vars_of(fusion.mmask); nb.dims = F.vars_of(fusion.nmask);
                }
                na.poly = Poly{ma}; nb.poly = Poly{mb};
                // a factor that is nothing but a small pre-evaluated sum: its kernel writes the column itself
                auto redirect = [&](Node &col, const Mono &m, int tensor) {
                    if (m.atoms.size() != 1 || m.c != 1.0 || w.inst[m.atoms[0]].op != I_LOAD) return false;
                    auto it = F.load_tensor.find(w.inst[m.atoms[0]].load);
                    if (it == F.load_tensor.end()) return false;
                    int writer = -1, n_writers = 0;
                    for (size_t q = 0; q < F.nodes.size(); ++q) if (F.nodes[q].tensor == it->second) { writer = (int)q; ++n_writers; }
                    if (n_writers != 1 || F.nodes[writer].kind != 0 || F.nodes[writer].dims != col.dims) return false;
                    // no other reader of that tensor in S
                    int readers = 0;
                    for (const Mono &o : S) for (int a : o.atoms) if (a == m.atoms[0]) ++readers;
                    if (readers != 1) return false;
                    F.nodes[writer].tensor = tensor; F.nodes[writer].col0 = col.col0;
                    return true;
                };
                if ((int)mi == t_mono || !redirect(na, ma, fusion.a_tensor)) F.nodes.push_back(na);
                if ((int)mi == t_mono || !redirect(nb, mb, fusion.b_tensor)) F.nodes.push_back(nb);
            }
            G.reqs.clear();                          // the contraction itself is the kernel now
            std::reverse(op.begin(), op.end()); std::reverse(imm.begin(), imm.end()); std::reverse(lds.begin(), lds.end());
            fusion.op = op; fusion.imm = imm; fusion.load = lds;
            fusion.on = true;
        }
    }

    // ---- layouts of the merged contractions ----
    // A group a few columns wider than 32 gives its single columns (plain and weighted sums of the streamed
    // operand) to passes of their own: those run at memory speed, and the rest fits the 32-column tile exactly
    // instead of padding every tile to the next width.
    for (size_t gi = 0, n_groups = F.groups.size(); gi < n_groups; ++gi) {
        auto width = [&](const Request &r) { int64_t wd = 1; for (int v = 0; v < TADP_MAX_VARS; ++v) if (r.nmask & (1u << v)) wd *= F.vext[v]; return wd; };
        int64_t total = 0;
        for (const Request &r : F.groups[gi].reqs) total += width(r);
        if (total <= 32 || total > 40) continue;
        // (an operand that is consecutive along its rows takes the streaming kernel, which holds 36 columns)
        {
            const TadpLoad &LA = w.loads[w.inst[F.groups[gi].a_inst].load];
            bool along_rows = false;
            for (int v = 0; v < TADP_MAX_VARS; ++v) if (!(F.groups[gi].kmask & (1u << v)) && std::abs(LA.coef[v]) == 1 && F.vext[v] > 1) along_rows = true;
            if (along_rows && total <= 36) continue;
        }
        for (size_t ri = 0; ri < F.groups[gi].reqs.size() && total > 32;) {
            const Request r = F.groups[gi].reqs[ri];
            const bool single = width(r) == 1 && (r.b_atoms.empty() || (r.b_atoms.size() == 1 && F.is_plain_load(r.b_atoms[0])));
            if (!single) { ++ri; continue; }
            Group G; G.a_inst = F.groups[gi].a_inst; G.kmask = F.groups[gi].kmask; G.reqs.push_back(r);
            F.groups[gi].reqs.erase(F.groups[gi].reqs.begin() + ri);
            F.groups.push_back(G);
            total -= 1;
        }
    }
    const int slot0 = p.n_args + 1 + (int)p.stages.size();
    const int max_aux = (p.opt.saved_forward ? TADP_F_SLOT : TADP_MAX_PTRS) - slot0;
    for (size_t gi = 0; gi < F.groups.size(); ++gi) {
        Group &G = F.groups[gi];
        if (G.reqs.empty()) continue;
        const uint32_t mmask = w.inst[G.a_inst].deps & ~G.kmask;
        const TadpLoad &LA = w.loads[w.inst[G.a_inst].load];
        // a single plain summation whose result depends on the outer variables through one affine row of the
        // operand: index the result by that row (sum_j G[beta - z, j] is a row sum of G, not one sum per (beta, z))
        if (G.reqs.size() == 1 && G.reqs[0].b_atoms.empty()) {
            int64_t gq = 0, lo = 0, hi = 0, klo = 0, khi = 0;
            bool boxed = true;                    // every row variable has a known range
            for (int v = 0; v < TADP_MAX_VARS; ++v) {
                if (!LA.coef[v]) continue;
                const int64_t span = (int64_t)LA.coef[v] * (F.vext[v] - 1), first = (int64_t)LA.coef[v] * F.vlo[v];
                if (G.kmask & (1u << v)) { klo += first + std::min<int64_t>(0, span); khi += first + std::max<int64_t>(0, span); }
                else {
                    gq = gcd64(gq, std::llabs((int64_t)LA.coef[v]));
                    lo += first + std::min<int64_t>(0, span); hi += first + std::max<int64_t>(0, span);
                    if (v >= g.n_outer && !F.can_sum[v] && w.vars[v].kind == 1) boxed = false;
                }
            }
            if (gq > 0) {
                // rows u with  base + gq u + (summed part)  inside the tensor
                int64_t u_min = ceil_div(-(int64_t)LA.base - klo, gq);
                int64_t u_max = floor_div((int64_t)LA.limit - 1 - LA.base - khi, gq);
                if (boxed) { u_min = std::max(u_min, ceil_div(lo, gq)); u_max = std::min(u_max, floor_div(hi, gq)); }
                const int64_t uext = u_max - u_min + 1;
                if (uext > 0 && (double)uext * 2 <= F.space(mmask)) { G.u_trick = true; G.u_g = gq; G.u0 = u_min; G.u_ext = uext; }
            }
        }
        if (G.u_trick) {
            Tensor T; T.cols = 1; T.elems = G.u_ext;
            F.tensors.push_back(T);
            G.t_tensor = (int)F.tensors.size() - 1;
            TadpLoad &L = w.loads[G.reqs[0].load_id];
            L = TadpLoad{};
            L.ptr = -1 - G.t_tensor; L.limit = to_i32(G.u_ext);
            int64_t base = -G.u0;
            for (int v = 0; v < TADP_MAX_VARS; ++v)
                if (LA.coef[v] && !(G.kmask & (1u << v))) L.coef[v] = to_i32(LA.coef[v] / G.u_g);
            L.base = to_i32(base);
            F.load_tensor[G.reqs[0].load_id] = G.t_tensor;
            continue;
        }
        int64_t cols = 0;
        for (Request &r : G.reqs) {
            r.col0 = cols; r.width = 1;
            for (int v = 0; v < TADP_MAX_VARS; ++v) if (r.nmask & (1u << v)) r.width = mul_ck(r.width, F.vext[v]);
            cols += r.width;
        }
        const bool direct = G.reqs.size() == 1 && (G.reqs[0].b_atoms.empty() || (G.reqs[0].b_atoms.size() == 1 && F.is_plain_load(G.reqs[0].b_atoms[0])));
        if (direct) {
            // the second operand is read where it lives; the result is indexed by the variables of both operands
            G.t_tensor = F.new_tensor(F.vars_of(mmask | G.reqs[0].nmask), 1);
            TadpLoad &L = w.loads[G.reqs[0].load_id];
            const Tensor &T = F.tensors[G.t_tensor];
            L = TadpLoad{};
            L.ptr = -1 - G.t_tensor; L.limit = to_i32(T.elems);
            int64_t base = 0;
            for (size_t d = 0; d < T.vars.size(); ++d) { L.coef[T.vars[d]] = to_i32(T.stride[d]); base -= T.stride[d] * F.vlo[T.vars[d]]; }
            L.base = to_i32(base);
            F.load_tensor[G.reqs[0].load_id] = G.t_tensor;
            continue;
        }
        // merged: X[summed variables, column], T[row variables, column]
        G.cols = cols;
        const int64_t padded = (cols + 3) / 4 * 4;          // rows of whole 16-byte pieces (copied as such by the kernels)
        G.x_tensor = F.new_tensor(F.vars_of(G.kmask), padded);
        G.t_tensor = F.new_tensor(F.vars_of(mmask), padded);
        for (Request &r : G.reqs) {
            // the block's own variables index its columns, last variable fastest
            std::vector<int> nvars = F.vars_of(r.nmask);
            std::vector<int64_t> cstride(nvars.size(), 1);
            for (int d = (int)nvars.size() - 2; d >= 0; --d) cstride[d] = cstride[d + 1] * F.vext[nvars[d + 1]];
            const Tensor &T = F.tensors[G.t_tensor];
            TadpLoad &L = w.loads[r.load_id];
            L = TadpLoad{};
            L.ptr = -1 - G.t_tensor; L.limit = to_i32(T.elems);
            int64_t base = r.col0;
            for (size_t d = 0; d < T.vars.size(); ++d) { L.coef[T.vars[d]] = to_i32(T.stride[d]); base -= T.stride[d] * F.vlo[T.vars[d]]; }
            for (size_t d = 0; d < nvars.size(); ++d) { L.coef[nvars[d]] = to_i32(L.coef[nvars[d]] + cstride[d]); base -= cstride[d] * F.vlo[nvars[d]]; }
            L.base = to_i32(base);
            F.load_tensor[r.load_id] = G.t_tensor;
            // the kernel that fills this block of X
            Node n; n.kind = 0; n.tensor = G.x_tensor; n.col0 = r.col0;
            n.dims = F.vars_of(G.kmask | r.nmask);
            Mono body; body.atoms = r.b_atoms;
            n.poly = Poly{body};
            n.group = (int)gi;
            F.nodes.push_back(n);
        }
    }
    for (size_t gi = 0; gi < F.groups.size(); ++gi) if (!F.groups[gi].reqs.empty()) { Node n; n.kind = 1; n.group = (int)gi; n.tensor = F.groups[gi].t_tensor; F.nodes.push_back(n); }
    if ((int)F.tensors.size() > max_aux) return false;

    // ---- auxiliary area: one slot and one 256-byte aligned region per tensor ----
    std::vector<int> slot_of(F.tensors.size());
    k.aux.clear();
    size_t cursor = 0;
    for (size_t t = 0; t < F.tensors.size(); ++t) {
        slot_of[t] = slot0 + (int)t;
        Kernel::Aux a; a.offset = cursor; a.bytes = size_t(F.tensors[t].elems) * 4; a.slot = slot_of[t];
        k.aux.push_back(a);
        cursor += (a.bytes + 255) & ~size_t(255);
    }
    k.aux_bytes = cursor;

    // ---- order: a kernel runs after the kernels that fill the tensors it reads ----
    auto reads_of_inst = [&](int root_inst, std::set<int> &out) {
        std::vector<int> st{root_inst}; std::set<int> seen;
        while (!st.empty()) {
            const int i = st.back(); st.pop_back();
            if (i < 0 || !seen.insert(i).second) continue;
            const Inst &in = w.inst[i];
            if (in.op == I_LOAD) { auto it = F.load_tensor.find(in.load); if (it != F.load_tensor.end()) out.insert(it->second); }
            st.push_back(in.a); st.push_back(in.b);
        }
    };
    std::vector<std::set<int>> node_reads(F.nodes.size());
    for (size_t n = 0; n < F.nodes.size(); ++n) {
        const Node &N = F.nodes[n];
        if (N.kind == 2) {}
        else if (N.kind == 0) { for (const Mono &m : N.poly) for (int a : m.atoms) reads_of_inst(a, node_reads[n]); }
        else {
            const Group &G = F.groups[N.group];
            reads_of_inst(G.a_inst, node_reads[n]);
            if (G.x_tensor >= 0) node_reads[n].insert(G.x_tensor);
            else for (const Request &r : G.reqs) for (int a : r.b_atoms) reads_of_inst(a, node_reads[n]);
        }
    }
    std::vector<int> order; std::vector<bool> done(F.nodes.size(), false);
    while (order.size() < F.nodes.size()) {
        bool progress = false;
        for (size_t n = 0; n < F.nodes.size(); ++n) {
            if (done[n]) continue;
            bool ready = true;
            for (int t : node_reads[n])
                for (size_t m = 0; m < F.nodes.size(); ++m) if (!done[m] && F.nodes[m].tensor == t) ready = false;
            if (!ready) continue;
            done[n] = true; order.push_back((int)n); progress = true;
        }
        if (!progress) return false;
    }

    // ---- build the kernels ----
    std::string text = "; factored: " + std::to_string(F.nodes.size()) + " auxiliary kernels, " + std::to_string(F.tensors.size()) + " auxiliary tensors\n";
    std::vector<Kernel> pre;
    for (int n : order) {
        const Node &N = F.nodes[n];
        Kernel ak;
        std::memset(&ak.prog, 0, sizeof ak.prog);
        ak.out_arg = -1; ak.access = -1; ak.out_aux = N.tensor;
        const Tensor &T = F.tensors[N.tensor];
        if (N.kind == 2) {
            // one output per element of the argument: the expression with its load read at the flat element index
            Gen g2(p, -1);
            Translator tr(w, g2, slot_of);
            g2.n_outer = 1; g2.kappa = 0;
            g2.new_var(0, T.elems);
            tr.flat_load = N.table_load;
            TadpProgram &ap = ak.prog;
            ap.outer_lo[0] = 0; ap.outer_ext[0] = to_i32(T.elems); ap.out_coef[0] = 1;
            ap.out_base = 0; ap.out_limit = to_i32(T.elems); ap.accumulate = 0; ap.write_only_live = 0;
            const int root2 = tr.run(N.table_inst);
            g2.lane_var = 0;
            emit_plain_kernel(g2, ak, root2, {}, {}, {}, false);
            text += "; function table -> tensor " + std::to_string(N.tensor) + "\n" + ak.listing;
        } else if (N.kind == 0) {
            Gen g2(p, -1);
            Translator tr(w, g2, slot_of);
            g2.n_outer = (int)N.dims.size(); g2.kappa = 0;
            TadpProgram &ap = ak.prog;
            // output offset: the tensor's own variables by their strides; a block of a merged tensor adds its
            // column variables (those of dims that are not variables of the tensor), last fastest
            std::vector<int64_t> ocoef(N.dims.size(), 0);
            int64_t obase = N.col0;
            int64_t cs = 1;
            for (int d = (int)N.dims.size() - 1; d >= 0; --d) {
                const int v = N.dims[d];
                auto it = std::find(T.vars.begin(), T.vars.end(), v);
                if (it != T.vars.end()) ocoef[d] = T.stride[it - T.vars.begin()];
                else { ocoef[d] = cs; cs *= F.vext[v]; }
            }
            for (size_t d = 0; d < N.dims.size(); ++d) {
                const int v = N.dims[d];
                const int nvid = g2.new_var(0, std::max<int64_t>(1, F.vext[v]));
                tr.var_map[v] = nvid;
                ap.outer_lo[d] = to_i32(F.vlo[v]); ap.outer_ext[d] = to_i32(std::max<int64_t>(1, F.vext[v]));
                ap.out_coef[d] = to_i32(ocoef[d]);
                obase -= ocoef[d] * F.vlo[v];
            }
            ap.out_base = to_i32(obase); ap.out_limit = to_i32(T.elems); ap.accumulate = 0; ap.write_only_live = 0;
            // summand, wrapped in the sums (as bound sums of the new kernel)
            int body = F.build_poly(N.poly);
            for (int v : N.sums) {
                Inst s; s.op = I_SUM; s.a = body; s.var = v; s.lo = F.vlo[v]; s.hi = F.vlo[v] + F.vext[v] - 1;
                s.deps = w.inst[body].deps & ~(1u << v);
                w.inst.push_back(s);                        // not interned: a private instance for the translation
                body = (int)w.inst.size() - 1;
            }
            // every load of the summand must stay inside its tensor over the whole box of this kernel (the box of a
            // masked index expression is a bounding box: points outside the image would read out of range)
            {
                uint32_t box = 0;
                for (int v : N.dims) box |= 1u << v;
                for (int v : N.sums) box |= 1u << v;
                std::vector<int> st{body}; std::set<int> seen;
                while (!st.empty()) {
                    const int i = st.back(); st.pop_back();
                    if (i < 0 || !seen.insert(i).second) continue;
                    const Inst &in = w.inst[i];
                    if (in.op == I_LOAD) {
                        const TadpLoad &L = w.loads[in.load];
                        int64_t lo = L.base, hi = L.base;
                        for (int v = 0; v < TADP_MAX_VARS; ++v) {
                            if (!L.coef[v]) continue;
                            if (!(box & (1u << v)) && w.vars[v].kind != 2) return false;
                            const int64_t first = (int64_t)L.coef[v] * F.vlo[v], span = (int64_t)L.coef[v] * (std::max<int64_t>(1, F.vext[v]) - 1);
                            lo += first + std::min<int64_t>(0, span); hi += first + std::max<int64_t>(0, span);
                        }
                        if (lo < 0 || hi >= L.limit) return false;
                    }
                    st.push_back(in.a); st.push_back(in.b);
                }
            }
            const int root2 = tr.run(body);
            if (g2.n_outer == 0) { g2.new_var(0, 1); g2.n_outer = 1; ap.outer_lo[0] = 0; ap.outer_ext[0] = 1; ap.out_coef[0] = 0; }
            // lanes along the variable with the smallest output stride
            int lane = g2.n_outer - 1;
            for (int d = 0; d < g2.n_outer; ++d) if (ap.out_coef[d] != 0 && (ap.out_coef[lane] == 0 || std::abs(ap.out_coef[d]) < std::abs(ap.out_coef[lane]))) lane = d;
            g2.lane_var = lane;
            emit_plain_kernel(g2, ak, root2, {}, {}, {}, false);
            text += "; auxiliary kernel -> tensor " + std::to_string(N.tensor) + "\n" + ak.listing;
        } else {
            const Group &G = F.groups[N.group];
            const TadpLoad &LA = w.loads[w.inst[G.a_inst].load];
            System s;
            s.loose_box = true;                            // offsets that leave a tensor: give the pass up, not the compilation
            const int nv = TADP_MAX_VARS + 1;              // the last one is the column index of a merged contraction
            s.vars.assign(nv, AVar{1, false});
            s.A.coef.assign(nv, 0); s.B.coef.assign(nv, 0); s.O.coef.assign(nv, 0);
            s.A.ptr = LA.ptr < 0 ? slot_of[-1 - LA.ptr] : LA.ptr; s.A.base = LA.base; s.A.limit = LA.limit;
            for (int v = 0; v < TADP_MAX_VARS; ++v) {
                if (!LA.coef[v] && !(G.kmask & (1u << v))) continue;
                s.vars[v] = AVar{std::max<int64_t>(0, F.vext[v]), (G.kmask & (1u << v)) != 0};
                s.A.coef[v] = LA.coef[v];
                s.A.base += (int64_t)LA.coef[v] * F.vlo[v];
            }
            s.O.ptr = slot_of[G.t_tensor]; s.O.limit = T.elems; s.O.base = 0;
            if (G.u_trick) {
                // rows u of the operand: A offset = base + g u + (summed part), all row variables collapse into u
                for (int v = 0; v < TADP_MAX_VARS; ++v) if (!(G.kmask & (1u << v))) { s.vars[v] = AVar{1, false}; s.A.coef[v] = 0; }
                s.A.base = LA.base;
                for (int v = 0; v < TADP_MAX_VARS; ++v) if (G.kmask & (1u << v)) s.A.base += (int64_t)LA.coef[v] * F.vlo[v];
                s.A.base += G.u_g * G.u0;
                s.vars[nv - 1] = AVar{G.u_ext, false};
                s.A.coef[nv - 1] = G.u_g; s.O.coef[nv - 1] = 1;
                s.B.ptr = -1;
            } else {
                for (size_t d = 0; d < T.vars.size(); ++d) s.O.coef[T.vars[d]] = T.stride[d];
                if (G.x_tensor >= 0) {
                    const Tensor &X = F.tensors[G.x_tensor];
                    s.B.ptr = slot_of[G.x_tensor]; s.B.limit = X.elems; s.B.base = 0;
                    for (size_t d = 0; d < X.vars.size(); ++d) s.B.coef[X.vars[d]] = X.stride[d];
                    s.vars[nv - 1] = AVar{G.cols, false};
                    s.B.coef[nv - 1] = 1; s.O.coef[nv - 1] = 1;
                } else if (G.reqs[0].b_atoms.empty()) s.B.ptr = -1;
                else {
                    const TadpLoad &LB = w.loads[w.inst[G.reqs[0].b_atoms[0]].load];
                    s.B.ptr = LB.ptr < 0 ? slot_of[-1 - LB.ptr] : LB.ptr; s.B.base = LB.base; s.B.limit = LB.limit;
                    for (int v = 0; v < TADP_MAX_VARS; ++v) {
                        if (!LB.coef[v]) continue;
                        if (s.vars[v].ext == 1 && !s.vars[v].reduce) s.vars[v] = AVar{std::max<int64_t>(0, F.vext[v]), false};
                        s.B.coef[v] = LB.coef[v];
                        s.B.base += (int64_t)LB.coef[v] * F.vlo[v];
                    }
                }
            }
            TadcProgram cp;
            if (!emit_program(s, 1.f, 0, true, false, cp, text)) return false;
            ak.contract.push_back(cp);
            ak.listing = "; contraction -> tensor " + std::to_string(N.tensor) + "\n";
            ak.vec = 0; ak.vec_u = 0;
        }
        pre.push_back(ak);
    }

    // ---- the kernel itself: the fused contraction, or the rewritten term under the loops that are left ----
    if (fusion.on) {
        System s;
        const int nv = TADP_MAX_VARS + 1;
        s.vars.assign(nv, AVar{1, false});
        s.A.coef.assign(nv, 0); s.B.coef.assign(nv, 0); s.O.coef.assign(nv, 0);
        const Tensor &TA = F.tensors[fusion.a_tensor], &TB = F.tensors[fusion.b_tensor];
        s.A.ptr = slot_of[fusion.a_tensor]; s.A.limit = TA.elems;
        s.B.ptr = slot_of[fusion.b_tensor]; s.B.limit = TB.elems;
        for (size_t d = 0; d < TA.vars.size(); ++d) { s.vars[TA.vars[d]] = AVar{F.vext[TA.vars[d]], false}; s.A.coef[TA.vars[d]] = TA.stride[d]; }
        for (size_t d = 0; d < TB.vars.size(); ++d) { s.vars[TB.vars[d]] = AVar{F.vext[TB.vars[d]], false}; s.B.coef[TB.vars[d]] = TB.stride[d]; }
        s.vars[nv - 1] = AVar{fusion.cols, true};
        s.A.coef[nv - 1] = 1; s.B.coef[nv - 1] = 1;
        s.O.base = prog.out_base; s.O.limit = prog.out_limit;
        for (int v = 0; v < g.n_outer; ++v) { s.O.coef[v] = prog.out_coef[v]; s.O.base += (int64_t)prog.out_coef[v] * F.vlo[v]; }
        TadcProgram cp;
        if (!emit_program(s, 1.f, prog.accumulate, false, false, cp, text)) return false;
        cp.n_epi = (int32_t)fusion.op.size();
        for (size_t e = 0; e < fusion.op.size(); ++e) {
            cp.epi_op[e] = fusion.op[e]; cp.epi_imm[e] = fusion.imm[e];
            if (fusion.load[e] >= 0) {
                const TadpLoad &L = w.loads[fusion.load[e]];
                cp.epi_ptr[e] = L.ptr; cp.epi_base[e] = to_i32((int64_t)L.base - prog.out_base);
            }
        }
        k.contract = {cp};
        k.vec = 0; k.vec_u = 0;
        char line[96];
        std::snprintf(line, sizeof line, "; the kernel is the contraction above with %d epilogue steps\n", cp.n_epi);
        k.listing = text + line;
        k.pre = pre;
        return true;
    }
    Gen g3(p, g.q);
    Translator tr(w, g3, slot_of);
    g3.n_outer = g.n_outer;
    for (int v = 0; v < g.n_outer; ++v) { g3.new_var(0, g.vars[v].ext); tr.var_map[v] = v; }
    std::vector<int> kept;                          // loop positions that stay
    for (int l = 0; l < g.kappa; ++l) if (std::find(summed.begin(), summed.end(), zvars[l]) == summed.end()) kept.push_back(l);
    g3.kappa = (int)kept.size();
    g3.zorder.resize(g3.kappa); g3.zpos.resize(g3.kappa);
    for (int l = 0; l < g3.kappa; ++l) { const int z = zvars[kept[l]]; tr.var_map[z] = g3.new_var(1, g.vars[z].ext); g3.zorder[l] = l; g3.zpos[l] = l; }
    auto map_row = [&](const TadpRow &r) {
        TadpRow n{}; n.den = r.den; n.c0 = r.c0;
        for (int v = 0; v < TADP_MAX_VARS; ++v) if (r.coef[v]) { if (tr.var_map[v] < 0) throw BadExpr("internal: bound row reads a summed variable"); n.coef[tr.var_map[v]] = r.coef[v]; }
        return n;
    };
    std::vector<std::vector<TadpRow>> lower3(g3.kappa), upper3(g3.kappa);
    for (int l = 0; l < g3.kappa; ++l) {
        for (const TadpRow &r : lower[kept[l]]) lower3[l].push_back(map_row(r));
        for (const TadpRow &r : upper[kept[l]]) upper3[l].push_back(map_row(r));
    }
    std::vector<TadpRow> guards3;
    for (const TadpRow &r : guards) guards3.push_back(map_row(r));
    const int root3 = tr.run(term);
    g3.stages_used = g.stages_used;
    // lanes: the caller's choice if that variable is still a loop of this kernel, else the variable along which
    // the output is contiguous
    int lane = -1;
    if (g.lane_var >= 0 && tr.var_map[g.lane_var] >= 0 && g.lane_var < g.n_outer + g.kappa) lane = tr.var_map[g.lane_var];
    if (lane < 0 || (g3.kappa == 0 && std::abs(prog.out_coef[lane]) != 1)) {
        lane = g.n_outer - 1;
        for (int v = 0; v < g.n_outer; ++v) if (prog.out_coef[v] != 0 && g3.vars[v].ext > 1 && (std::abs(prog.out_coef[v]) < std::abs(prog.out_coef[lane]) || prog.out_coef[lane] == 0)) lane = v;
    }
    g3.lane_var = lane;
    Kernel main = k;
    main.pre.clear(); main.contract.clear(); main.ew.clear(); main.line.clear();
    emit_plain_kernel(g3, main, root3, lower3, upper3, guards3, allow_split);
    k.prog = main.prog; k.vec = main.vec; k.vec_u = main.vec_u; k.rich = main.rich; k.contract = main.contract; k.ew = main.ew; k.line = main.line;
    k.listing = text + main.listing;
    k.pre = pre;
    return true;
}

bool try_factoring(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
                   const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards)
{
    const Kernel saved = k;
    try {
        if (factor_kernel(g, k, root, scale, allow_split, lower, upper, guards)) return true;
    } catch (const Unsupported &) {
    } catch (const Overflow &) {
    }
    k = saved;                  // too many variables, loads or temporaries somewhere: the kernel stays as it was
    return false;
}

}  // namespace tad

// Printer of an expression and of its derived derivative expressions in the notation of Sec. 6:
//   f[i; j] = exp (-sum{k}_0^4 (...))
//   dx[dx_0; dx_1] = if {conditions} then (sum{dx_z1}_lo^hi (sum{dx_z0}_lo^hi (term))) else (0)
// The derivative is read off the plan: the index transform alpha = I beta + K z (Sec. 5.1) written out per index
// position, the conditions of the cokernel and of divisibility, the bound rows of Sec. 4.2 as max [..] / min [..]
// of affine forms, and the term as the adjoint carried from the root to the leaf by the rules of Sec. 2
// (every step multiplies the adjoint by the local derivative).  Sums on the way to the leaf are liberated
// (Sec. 5.2): their index is replaced by its affine form; sums inside any other operand keep their own index.
// Host only.
#include <algorithm>
#include <cstdio>
#include <functional>
#include <map>
#include <string>
#include <vector>

#include "../../include/tad.h"
#include "plan.h"

namespace tad {

namespace {

struct Rat { int64_t n = 0, d = 1; };
Rat norm(Rat r)
{
    if (r.d < 0) { r.n = -r.n; r.d = -r.d; }
    const int64_t g = gcd64(r.n < 0 ? -r.n : r.n, r.d);
    if (g > 1) { r.n /= g; r.d /= g; }
    if (r.n == 0) r.d = 1;
    return r;
}
Rat add(Rat a, Rat b) { return norm(Rat{a.n * b.d + b.n * a.d, a.d * b.d}); }
Rat mul(Rat a, Rat b) { return norm(Rat{a.n * b.n, a.d * b.d}); }

// constant + sum of coefficient * name; names keep the order of first use
struct Affine {
    Rat c;
    std::vector<std::pair<std::string, Rat>> terms;
    void add_term(const std::string &name, Rat k)
    {
        if (k.n == 0) return;
        for (auto &t : terms) if (t.first == name) { t.second = add(t.second, k); return; }
        terms.push_back({name, norm(k)});
    }
    void add_affine(const Affine &o, Rat k)
    {
        c = add(c, mul(o.c, k));
        for (const auto &t : o.terms) add_term(t.first, mul(t.second, k));
    }
    bool constant() const { for (const auto &t : terms) if (t.second.n != 0) return false; return true; }
};

std::string num(int64_t v) { return std::to_string(v); }
std::string rat(Rat r) { return r.d == 1 ? num(r.n) : "(" + num(r.n) + " / " + num(r.d) + ")"; }

// "-2 + dd_0", "dd_0 + -dd_z1", "2 * i + k"
std::string text(const Affine &a)
{
    std::string out;
    auto piece = [&](const std::string &s) { out += out.empty() ? s : " + " + s; };
    if (a.c.n != 0) piece(rat(a.c));
    for (const auto &t : a.terms) {
        const Rat k = t.second;
        if (k.n == 0) continue;
        if (k.d == 1 && k.n == 1) piece(t.first);
        else if (k.d == 1 && k.n == -1) piece("-" + t.first);
        else piece(rat(k) + " * " + t.first);
    }
    return out.empty() ? "0" : out;
}

// all coefficients times m, as integers (m a common multiple of the denominators)
Affine scaled(const Affine &a, int64_t m)
{
    Affine r;
    r.add_affine(a, Rat{m, 1});
    return r;
}
int64_t common_den(const Affine &a)
{
    int64_t l = a.c.d;
    for (const auto &t : a.terms) l = l / gcd64(l, t.second.d) * t.second.d;
    return l;
}

struct Printer {
    const tad_plan &p;
    std::vector<std::string> arg_names, idx_names;
    std::map<int, Affine> subst;            // alpha_hat position -> its affine form (derivatives only)

    std::string constant(double v) const
    {
        char b[64];
        if (v == (double)(int64_t)v && v > -1e15 && v < 1e15) std::snprintf(b, sizeof b, "%lld", (long long)v);
        else std::snprintf(b, sizeof b, "%.9g", v);
        return b;
    }
    // index list of a load: A alpha_hat + offset with bound positions by name, the others substituted
    std::string indices(int q, uint32_t bound) const
    {
        const int n_idx = p.n_out + p.n_sum, rank = (int)p.accOff[q].size();
        std::string out;
        for (int r = 0; r < rank; ++r) {
            Affine a;
            a.c = Rat{p.accOff[q][r], 1};
            for (int d = 0; d < n_idx; ++d) {
                const int64_t c = p.accA[q][size_t(r) * n_idx + d];
                if (!c) continue;
                const bool is_bound = d >= p.n_out && (bound & (1u << (d - p.n_out)));
                auto it = subst.find(d);
                if (is_bound || it == subst.end()) a.add_term(idx_names[d], Rat{c, 1});
                else a.add_affine(it->second, Rat{c, 1});
            }
            out += (r ? "; " : "") + text(a);
        }
        return out;
    }
    bool atom(int n) const { const int op = p.nodes[n].op; return op == TAD_OP_CONST || op == TAD_OP_LOAD; }
    // a value as an operand of *, ** or a unary minus: compound values in parentheses
    std::string operand(int n, uint32_t bound) const
    {
        const int op = p.nodes[n].op;
        const std::string s = value(n, bound);
        if (atom(n) || op == TAD_OP_ADD || op == TAD_OP_SUB || (op >= TAD_OP_EXP && op <= TAD_OP_COSH)) return s;   // (a + b) carries its own
        if (op == TAD_OP_SUM || op == TAD_OP_POWI) return s;
        return "(" + s + ")";
    }
    std::string value(int n, uint32_t bound) const
    {
        const NodeH &nd = p.nodes[n];
        static const char *fn[] = {"exp", "log", "sin", "cos", "tanh", "sinh", "cosh"};
        switch (nd.op) {
        case TAD_OP_CONST: return constant(nd.imm);
        case TAD_OP_LOAD: return arg_names[p.accArg[nd.access]] + "[" + indices(nd.access, bound) + "]";
        case TAD_OP_NEG: return "-" + operand(nd.in0, bound);
        case TAD_OP_ADD: return "(" + value(nd.in0, bound) + " + " + value(nd.in1, bound) + ")";
        case TAD_OP_SUB: return "(" + value(nd.in0, bound) + " - " + operand(nd.in1, bound) + ")";
        case TAD_OP_MUL: return operand(nd.in0, bound) + " * " + operand(nd.in1, bound);
        case TAD_OP_DIV: return operand(nd.in0, bound) + " / " + operand(nd.in1, bound);
        case TAD_OP_POWI: return operand(nd.in0, bound) + " ** " + (nd.ipow < 0 ? "(" + num(nd.ipow) + ")" : num(nd.ipow));
        case TAD_OP_SUM:
            return "sum{" + idx_names[nd.sum_idx] + "}_" + num(nd.sum_lo) + "^" + num(nd.sum_hi) + " (" +
                   value(nd.in0, bound | (1u << (nd.sum_idx - p.n_out))) + ")";
        default:
            if (nd.op >= TAD_OP_EXP && nd.op <= TAD_OP_COSH) return std::string(fn[nd.op - TAD_OP_EXP]) + " (" + value(nd.in0, bound) + ")";
            return "?";
        }
    }
    std::string derivative(int q);
};

std::string Printer::derivative(int q)
{
    const AccessPlan &ap = p.access[q];
    const std::string x = arg_names[ap.arg], dx = "d" + x;
    auto beta = [&](int b) { return dx + "_" + num(b); };
    auto zname = [&](int col) { return dx + "_z" + num(col); };           // named by kernel column, as in Sec. 6
    // For the text a kernel coordinate runs in the direction that makes the last non-zero entry of its kernel
    // vector positive (z and -z describe the same set; the listing of Sec. 6 uses this direction)
    std::vector<int64_t> zsign(ap.kappa, 1);
    for (int m = 0; m < ap.kappa; ++m)
        for (int c = ap.n - 1; c >= 0; --c)
            if (ap.V(c, ap.R + m) != 0) { zsign[m] = ap.V(c, ap.R + m) < 0 ? -1 : 1; break; }
    // x'_j = (U_R (beta - o))_j / alpha_j
    std::vector<Affine> xp(ap.R);
    auto u_row = [&](int j) {
        Affine a;
        for (int b = 0; b < ap.rank; ++b) {
            a.add_term(beta(b), Rat{ap.U(j, b), 1});
            a.c = add(a.c, Rat{-ap.U(j, b) * ap.off[b], 1});
        }
        return a;
    };
    for (int j = 0; j < ap.R; ++j) { xp[j].add_affine(u_row(j), Rat{1, ap.inv[j]}); }
    // alpha_hat = V (x', z): the index transform of Sec. 5.1, per position
    subst.clear();
    for (int c = 0; c < ap.n; ++c) {
        Affine a;
        for (int j = 0; j < ap.R; ++j) a.add_affine(xp[j], Rat{ap.V(c, j), 1});
        for (int m = 0; m < ap.kappa; ++m) a.add_term(zname(m), Rat{ap.V(c, ap.R + m) * zsign[m], 1});
        subst[ap.idx_pos[c]] = a;
    }
    // ---- the term: adjoints from the root down to the loads of this index expression ----
    const int root = (int)p.nodes.size() - 1;
    std::vector<std::vector<std::pair<int, int>>> parents(p.nodes.size());   // (parent, which operand)
    for (int n = 0; n <= root; ++n) {
        if (!p.nodes[n].reachable) continue;
        if (p.nodes[n].in0 >= 0) parents[p.nodes[n].in0].push_back({n, 0});
        if (p.nodes[n].in1 >= 0) parents[p.nodes[n].in1].push_back({n, 1});
    }
    auto factor = [](const std::string &s) { return !s.empty() && s[0] == '-' ? "(" + s + ")" : s; };
    std::function<std::string(int)> adjoint = [&](int n) -> std::string {
        if (n == root) {
            std::string idx;
            for (int d = 0; d < p.n_out; ++d) idx += (d ? "; " : "") + text(subst.count(d) ? subst[d] : Affine{});
            return "df[" + idx + "]";
        }
        std::vector<std::string> parts;
        for (const auto &pr : parents[n]) {
            const NodeH &pn = p.nodes[pr.first];
            const std::string a = adjoint(pr.first);
            const std::string u = pn.in0 >= 0 ? operand(pn.in0, 0) : "", v = pn.in1 >= 0 ? operand(pn.in1, 0) : "";
            std::string t;
            switch (pn.op) {
            case TAD_OP_NEG: t = "-(" + a + ")"; break;
            case TAD_OP_ADD: case TAD_OP_SUM: t = a; break;
            case TAD_OP_SUB: t = pr.second == 0 ? a : "-(" + a + ")"; break;
            case TAD_OP_MUL: t = pr.second == 0 ? factor(a) + " * " + v : u + " * " + factor(a); break;
            case TAD_OP_DIV: t = pr.second == 0 ? factor(a) + " / " + v : "-(" + factor(a) + " * " + u + " / " + v + " ** 2)"; break;
            case TAD_OP_POWI: t = factor(a) + " * " + num(pn.ipow) + " * " + u + " ** (" + num(pn.ipow) + " - 1)"; break;
            case TAD_OP_EXP: t = factor(a) + " * exp (" + value(pn.in0, 0) + ")"; break;
            case TAD_OP_LOG: t = factor(a) + " / " + u; break;
            case TAD_OP_SIN: t = factor(a) + " * cos (" + value(pn.in0, 0) + ")"; break;
            case TAD_OP_COS: t = "-(" + factor(a) + " * sin (" + value(pn.in0, 0) + "))"; break;
            case TAD_OP_TANH: t = factor(a) + " * (1 - tanh (" + value(pn.in0, 0) + ") ** 2)"; break;
            case TAD_OP_SINH: t = factor(a) + " * cosh (" + value(pn.in0, 0) + ")"; break;
            case TAD_OP_COSH: t = factor(a) + " * sinh (" + value(pn.in0, 0) + ")"; break;
            default: t = "?"; break;
            }
            parts.push_back(t);
        }
        if (parts.empty()) return "0";
        if (parts.size() == 1) return parts[0];
        std::string s = "(" + parts[0];
        for (size_t i = 1; i < parts.size(); ++i) s += " + " + parts[i];
        return s + ")";
    };
    std::vector<std::string> leaves;
    for (int n = 0; n <= root; ++n)
        if (p.nodes[n].reachable && p.nodes[n].op == TAD_OP_LOAD && p.nodes[n].access == q) leaves.push_back(adjoint(n));
    std::string term = leaves.empty() ? "0" : leaves[0];
    for (size_t i = 1; i < leaves.size(); ++i) term += " + " + leaves[i];
    term = "(" + term + ")";
    // ---- a bound row as text: (c0 + cx . x' + cz . z) / den with true ceiling / floor when it does not divide ----
    auto row_text = [&](const BoundRowH &r, bool upper, bool bare, int64_t sign) {
        Affine a;
        a.c = Rat{r.c0, 1};
        for (int j = 0; j < ap.R && j < (int)r.cx.size(); ++j) a.add_affine(xp[j], Rat{r.cx[j], 1});
        for (size_t m = 0; m < r.cz.size(); ++m) a.add_term(zname(ap.zorder[m]), Rat{r.cz[m] * zsign[ap.zorder[m]], 1});
        Affine b;
        b.add_affine(a, Rat{sign, r.den});
        const int64_t l = common_den(b);
        if (bare || l == 1) return text(b);
        return std::string(upper ? "floor" : "ceil") + " ((" + text(scaled(b, l)) + ") / " + num(l) + ")";
    };
    auto range_text = [&](const std::vector<BoundRowH> &rows, bool upper, int64_t sign) {
        std::string s;
        if (rows.size() == 1) s = row_text(rows[0], upper, false, sign);
        else {
            s = upper ? "min [" : "max [";
            for (size_t i = 0; i < rows.size(); ++i) s += (i ? "; " : "") + row_text(rows[i], upper, false, sign);
            s += "]";
        }
        const bool plain = s.find(' ') == std::string::npos;
        return plain ? s : "(" + s + ")";
    };
    // ---- loops, outermost first ----
    std::string body = term;
    for (int l = ap.kappa - 1; l >= 0; --l) {
        // a reversed coordinate runs from minus the upper rows to minus the lower rows
        const bool rev = zsign[ap.zorder[l]] < 0;
        body = "sum{" + zname(ap.zorder[l]) + "}_" + range_text(rev ? ap.upper[l] : ap.lower[l], false, rev ? -1 : 1) + "^" +
               range_text(rev ? ap.lower[l] : ap.upper[l], true, rev ? -1 : 1) + " (" + body + ")";
    }
    // ---- conditions: cokernel rows, divisibility (the reading that keeps it), guards ----
    std::vector<std::string> conds;
    for (int j = ap.R; j < ap.rank; ++j) {
        Affine a = u_row(j);
        for (const auto &t : a.terms) if (t.second.n != 0) { if (t.second.n < 0) a = scaled(a, -1); break; }
        conds.push_back(text(a) + " = 0");
    }
    for (int j = 0; j < ap.R; ++j) if (ap.inv[j] > 1) conds.push_back("(" + text(u_row(j)) + ") mod " + num(ap.inv[j]) + " = 0");
    for (const BoundRowH &gr : ap.guards) {
        BoundRowH numerator = gr;
        numerator.den = 1;
        Affine a;
        a.c = Rat{gr.c0, 1};
        for (int j = 0; j < ap.R && j < (int)gr.cx.size(); ++j) a.add_affine(xp[j], Rat{gr.cx[j], 1});
        // (a guard that every element of the tensor satisfies is not a condition: interval arithmetic over its shape)
        const Affine g = scaled(a, common_den(a));
        Rat top = g.c;
        for (int b = 0; b < ap.rank; ++b)
            for (const auto &t : g.terms)
                if (t.first == beta(b) && t.second.n > 0) top = add(top, mul(t.second, Rat{p.arg_shape[ap.arg][b] - 1, 1}));
        if (top.n <= 0) continue;
        conds.push_back(text(g) + " <= 0");
    }
    std::string lhs = dx + "[";
    for (int b = 0; b < ap.rank; ++b) lhs += (b ? "; " : "") + beta(b);
    lhs += "] = ";
    if (conds.empty()) return lhs + body;
    std::string c = conds[0];
    for (size_t i = 1; i < conds.size(); ++i) c += "; " + conds[i];
    return lhs + "if {" + c + "} then (" + body + ") else (0)";
}

}  // namespace

// which = -1: the expression itself; which = q >= 0: the derivative through index expression q
std::string print_expression(const tad_plan &p, int which, const char *const *arg_names, const char *const *idx_names)
{
    Printer pr{p, {}, {}, {}};
    for (int a = 0; a < p.n_args; ++a) pr.arg_names.push_back(arg_names && arg_names[a] ? arg_names[a] : "x" + std::to_string(a));
    const int n_idx = p.n_out + p.n_sum;
    for (int d = 0; d < n_idx; ++d) {
        if (idx_names && idx_names[d]) pr.idx_names.push_back(idx_names[d]);
        else pr.idx_names.push_back(d < 18 ? std::string(1, char('i' + d)) : "i" + std::to_string(d));
    }
    if (which < 0) {
        std::string lhs = "f[";
        for (int d = 0; d < p.n_out; ++d) lhs += (d ? "; " : "") + pr.idx_names[d];
        return lhs + "] = " + pr.value((int)p.nodes.size() - 1, 0);
    }
    if (which >= (int)p.access.size() || !p.access[which].used) return "";
    return pr.derivative(which);
}

}  // namespace tad

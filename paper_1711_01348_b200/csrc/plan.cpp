// Expression validation and the integer analysis of every index expression (host only).
#include "plan.h"

#include <algorithm>
#include <cstring>
#include <tuple>

namespace tad {

namespace {

int arity(int op)
{
    switch (op) {
    case TAD_OP_CONST: case TAD_OP_LOAD: return 0;
    case TAD_OP_ADD: case TAD_OP_SUB: case TAD_OP_MUL: case TAD_OP_DIV: return 2;
    default: return 1;
    }
}

}  // namespace

void build_expression(tad_plan &p, const tad_expr *e, const tad_options *opt)
{
    if (!e) throw InvalidArg("expr is NULL");
    if (opt) {
        p.opt = *opt;
        for (int i = 0; i < 6; ++i) if (opt->reserved[i] != 0) throw InvalidArg("tad_options.reserved must be zero");
    }
    if (e->n_out_dims < 1 || e->n_sum_idx < 0 || e->n_args < 0 || e->n_access < 0 || e->n_nodes < 1)
        throw InvalidArg("negative or zero count in tad_expr");
    if (!e->out_shape || !e->nodes || (e->n_args && (!e->arg_rank || !e->arg_shape)) || (e->n_access && !e->access))
        throw InvalidArg("NULL array in tad_expr");
    const int n_idx = e->n_out_dims + e->n_sum_idx;
    if (n_idx > TAD_MAX_IDX) throw Unsupported("more than TAD_MAX_IDX output + sum indices");
    // pointer slots: the arguments, df, and the saved forward output when the plan reads it
    if (e->n_args + 1 + ((opt && opt->saved_forward) ? 1 : 0) > TADP_MAX_PTRS) throw Unsupported("too many arguments");
    p.n_out = e->n_out_dims; p.n_sum = e->n_sum_idx; p.n_args = e->n_args;
    p.out_shape.assign(e->out_shape, e->out_shape + e->n_out_dims);
    p.out_elems = 1;
    for (int64_t s : p.out_shape) {
        if (s < 1) throw InvalidArg("output extent < 1");
        p.out_elems = mul_ck(p.out_elems, s);
    }
    if (p.out_elems >= (int64_t(1) << 31)) throw Overflow();
    p.arg_shape.resize(p.n_args);
    p.arg_elems.resize(p.n_args);
    for (int a = 0; a < p.n_args; ++a) {
        int r = e->arg_rank[a];
        if (r < 1 || r > TAD_MAX_RANK) throw Unsupported("argument rank outside 1..TAD_MAX_RANK");
        if (!e->arg_shape[a]) throw InvalidArg("NULL argument shape");
        p.arg_shape[a].assign(e->arg_shape[a], e->arg_shape[a] + r);
        int64_t n = 1;
        for (int64_t s : p.arg_shape[a]) { if (s < 1) throw InvalidArg("argument extent < 1"); n = mul_ck(n, s); }
        if (n >= (int64_t(1) << 31)) throw Overflow();
        p.arg_elems[a] = n;
    }
    p.accA.resize(e->n_access); p.accOff.resize(e->n_access); p.accArg.resize(e->n_access);
    for (int q = 0; q < e->n_access; ++q) {
        const tad_access &a = e->access[q];
        if (a.arg < 0 || a.arg >= p.n_args) throw BadExpr("index expression names a missing argument");
        if (!a.A || !a.offset) throw InvalidArg("NULL matrix or offset in an index expression");
        int r = (int)p.arg_shape[a.arg].size();
        p.accArg[q] = a.arg;
        p.accA[q].assign(a.A, a.A + size_t(r) * n_idx);
        p.accOff[q].assign(a.offset, a.offset + r);
    }
    // nodes
    p.nodes.resize(e->n_nodes);
    p.sum_lo.assign(p.n_sum, 0); p.sum_hi.assign(p.n_sum, -1); p.sum_node.assign(p.n_sum, -1);
    for (int i = 0; i < e->n_nodes; ++i) {
        const tad_node &s = e->nodes[i];
        NodeH &d = p.nodes[i];
        d.op = s.op; d.in0 = s.in0; d.in1 = s.in1; d.access = s.access; d.ipow = s.ipow;
        d.sum_idx = s.sum_idx; d.sum_lo = s.sum_lo; d.sum_hi = s.sum_hi; d.imm = s.imm;
        if (s.op < TAD_OP_CONST || s.op > TAD_OP_SUM) throw BadExpr("unknown operation");
        int ar = arity(s.op);
        if (ar >= 1 && (s.in0 < 0 || s.in0 >= i)) throw BadExpr("operand 0 is not an earlier node");
        if (ar >= 2 && (s.in1 < 0 || s.in1 >= i)) throw BadExpr("operand 1 is not an earlier node");
        if (ar < 1) d.in0 = -1;
        if (ar < 2) d.in1 = -1;
        if (s.op == TAD_OP_LOAD && (s.access < 0 || s.access >= e->n_access)) throw BadExpr("load names a missing index expression");
        if (s.op == TAD_OP_SUM) {
            if (s.sum_idx < p.n_out || s.sum_idx >= n_idx) throw BadExpr("sum index outside the sum-index range");
            if (s.sum_hi < s.sum_lo) throw BadExpr("empty sum range");
            if (s.sum_hi - s.sum_lo >= (int64_t(1) << 30) || std::llabs(s.sum_lo) >= (int64_t(1) << 30)) throw Overflow();
        }
        if (s.op == TAD_OP_POWI && (s.ipow > 64 || s.ipow < -64)) throw Unsupported("|exponent| > 64");
    }
    // reachability and enclosing-sum sets, parents before children (operands have smaller ids)
    const int root = e->n_nodes - 1;
    std::vector<bool> scope_set(e->n_nodes, false);
    p.nodes[root].reachable = true; scope_set[root] = true; p.nodes[root].scope = 0;
    for (int i = root; i >= 0; --i) {
        NodeH &nd = p.nodes[i];
        if (!nd.reachable) continue;
        uint32_t child_scope = nd.scope;
        if (nd.op == TAD_OP_SUM) {
            int s = nd.sum_idx - p.n_out;
            if (p.sum_node[s] >= 0) throw Unsupported("a sum index is used by more than one sum node");
            if (nd.scope & (1u << s)) throw BadExpr("sum nested inside a sum over the same index");
            p.sum_node[s] = i; p.sum_lo[s] = nd.sum_lo; p.sum_hi[s] = nd.sum_hi;
            child_scope |= 1u << s;
        }
        for (int c : {nd.in0, nd.in1}) {
            if (c < 0) continue;
            NodeH &ch = p.nodes[c];
            if (scope_set[c] && ch.scope != child_scope && ch.op != TAD_OP_CONST)
                throw Unsupported("a node is used under two different sets of enclosing sums");
            ch.reachable = true; scope_set[c] = true; ch.scope = child_scope;
        }
    }
    // per index expression: one enclosing-sum set, indices only of enclosing sums, reads inside the shape
    p.access.assign(e->n_access, AccessPlan());
    for (int i = 0; i <= root; ++i) {
        const NodeH &nd = p.nodes[i];
        if (!nd.reachable || nd.op != TAD_OP_LOAD) continue;
        AccessPlan &ap = p.access[nd.access];
        if (ap.used && ap.scope != nd.scope)
            throw Unsupported("one index expression is read under two different sets of enclosing sums");
        ap.used = true; ap.scope = nd.scope;
    }
    for (int q = 0; q < e->n_access; ++q) {
        AccessPlan &ap = p.access[q];
        ap.arg = p.accArg[q];
        ap.rank = (int)p.arg_shape[ap.arg].size();
        if (!ap.used) continue;
        for (int r = 0; r < ap.rank; ++r) {
            int64_t lo = p.accOff[q][r], hi = p.accOff[q][r];
            for (int d = 0; d < n_idx; ++d) {
                int64_t c = p.accA[q][size_t(r) * n_idx + d];
                if (c == 0) continue;
                int64_t dlo, dhi;
                if (d < p.n_out) { dlo = 0; dhi = p.out_shape[d] - 1; }
                else {
                    int s = d - p.n_out;
                    if (!(ap.scope & (1u << s))) throw BadExpr("index expression uses a sum index outside that sum");
                    dlo = p.sum_lo[s]; dhi = p.sum_hi[s];
                }
                lo = add_ck(lo, mul_ck(c, c > 0 ? dlo : dhi));
                hi = add_ck(hi, mul_ck(c, c > 0 ? dhi : dlo));
            }
            if (lo < 0 || hi >= p.arg_shape[ap.arg][r])
                throw OutOfRange("index expression " + std::to_string(q) + " leaves dimension " + std::to_string(r) +
                                 " of its argument: reaches [" + std::to_string(lo) + ", " + std::to_string(hi) + "]");
        }
    }
}

namespace {

// value range of  c0 + sum_j c[j] * v_j  for v in the inclusive box
void affine_range(int64_t c0, const std::vector<int64_t> &c, const std::vector<int64_t> &lo,
                  const std::vector<int64_t> &hi, int64_t &mn, int64_t &mx)
{
    mn = mx = c0;
    for (size_t j = 0; j < c.size(); ++j) {
        if (c[j] == 0) continue;
        mn = add_ck(mn, mul_ck(c[j], c[j] > 0 ? lo[j] : hi[j]));
        mx = add_ck(mx, mul_ck(c[j], c[j] > 0 ? hi[j] : lo[j]));
    }
}

void reduce_row(BoundRowH &r)
{
    int64_t g = gcd64(r.den, r.c0);
    for (int64_t v : r.cx) g = gcd64(g, v);
    for (int64_t v : r.cz) g = gcd64(g, v);
    if (g > 1) {
        r.den /= g; r.c0 /= g;
        for (int64_t &v : r.cx) v /= g;
        for (int64_t &v : r.cz) v /= g;
    }
}

bool same_row(const BoundRowH &a, const BoundRowH &b)
{
    return a.den == b.den && a.c0 == b.c0 && a.cx == b.cx && a.cz == b.cz;
}

}  // namespace

// Computes the bound rows of the kernel coordinates for the loop order ap.zorder
// (Sec. 5.1: the box constraints written as  K z >= lo - I beta,  -K z >= I beta - hi,
// then Fourier-Motzkin elimination, innermost loop first).
void compute_bounds(AccessPlan &ap)
{
    const int n = ap.n, R = ap.R, kap = ap.kappa;
    ap.lower.assign(kap, {}); ap.upper.assign(kap, {}); ap.guards.clear();
    Mat C(2 * n, std::max(kap, 1));
    if (kap == 0) C = Mat(2 * n, 0);
    for (int d = 0; d < n; ++d)
        for (int l = 0; l < kap; ++l) {
            int64_t k = ap.V(d, R + ap.zorder[l]);
            C(d, l) = k;
            C(n + d, l) = neg_ck(k);
        }
    std::vector<int> order;
    for (int l = kap - 1; l >= 0; --l) order.push_back(l);
    FmResult fm = fourier_motzkin(C, order, TAD_MAX_BOUND_ROWS);
    // right-hand sides over x':  b_d = lo_d - (V_R x')_d ,  b_{n+d} = (V_R x')_d - hi_d
    auto convert = [&](const std::vector<int64_t> &bcoef, BoundRowH &row) {
        row.c0 = 0; row.cx.assign(R, 0);
        for (int d = 0; d < n; ++d) {
            int64_t bl = bcoef[d], bh = bcoef[n + d];
            row.c0 = add_ck(row.c0, sub_ck(mul_ck(bl, ap.box_lo[d]), mul_ck(bh, ap.box_hi[d])));
            for (int j = 0; j < R; ++j)
                row.cx[j] = add_ck(row.cx[j], mul_ck(sub_ck(bh, bl), ap.V(d, j)));
        }
    };
    for (int l = 0; l < kap; ++l)
        for (int side = 0; side < 2; ++side) {
            const std::vector<FmBound> &src = side ? fm.upper[l] : fm.lower[l];
            std::vector<BoundRowH> &dst = side ? ap.upper[l] : ap.lower[l];
            if (src.empty()) throw Unsupported("a kernel coordinate is unbounded on one side");
            for (const FmBound &b : src) {
                BoundRowH row;
                convert(b.bcoef, row);
                row.den = b.den;
                row.cz.assign(kap, 0);
                for (int m = 0; m < kap; ++m) {
                    row.cz[m] = b.zcoef[m];
                    if (m >= l && b.zcoef[m] != 0) throw Unsupported("internal: bound row reads an inner loop");
                }
                reduce_row(row);
                bool dup = false;
                for (const BoundRowH &o : dst) if (same_row(o, row)) dup = true;
                if (!dup) dst.push_back(row);
            }
        }
    for (const std::vector<int64_t> &f : fm.feas) {
        BoundRowH row;
        convert(f, row);
        row.den = 1; row.cz.assign(kap, 0);
        bool constant = true;
        for (int64_t v : row.cx) if (v != 0) constant = false;
        if (constant) {
            if (row.c0 > 0) throw BadExpr("internal: the index box is empty");
            continue;                                  // constant row that holds
        }
        int64_t g = 0;
        for (int64_t v : row.cx) g = gcd64(g, v);
        if (g > 1) {                                   // sum cx x' <= -c0 over integers: tighten
            for (int64_t &v : row.cx) v /= g;
            row.c0 = neg_ck(floor_div(neg_ck(row.c0), g));
        }
        bool dup = false;
        for (const BoundRowH &o : ap.guards) if (same_row(o, row)) dup = true;
        if (!dup) ap.guards.push_back(row);
    }
}

void analyse_access(tad_plan &p, int q)
{
    AccessPlan &ap = p.access[q];
    const int n_idx = p.n_out + p.n_sum;
    ap.idx_pos.clear();
    for (int d = 0; d < n_idx; ++d)
        if (d < p.n_out || (ap.scope & (1u << (d - p.n_out)))) ap.idx_pos.push_back(d);
    ap.n = (int)ap.idx_pos.size();
    ap.A = Mat(ap.rank, ap.n);
    ap.off = p.accOff[q];
    ap.box_lo.resize(ap.n); ap.box_hi.resize(ap.n);
    for (int c = 0; c < ap.n; ++c) {
        int d = ap.idx_pos[c];
        for (int r = 0; r < ap.rank; ++r) ap.A(r, c) = p.accA[q][size_t(r) * n_idx + d];
        if (d < p.n_out) { ap.box_lo[c] = 0; ap.box_hi[c] = p.out_shape[d] - 1; }
        else { ap.box_lo[c] = p.sum_lo[d - p.n_out]; ap.box_hi[c] = p.sum_hi[d - p.n_out]; }
    }
    Smith sm = smith_normal_form(ap.A);
    ap.U = sm.U; ap.V = sm.V; ap.R = sm.rank; ap.kappa = ap.n - sm.rank;
    if (ap.kappa > TAD_MAX_KAPPA) throw Unsupported("kernel dimension > TAD_MAX_KAPPA");
    ap.inv.resize(ap.R);
    ap.masked = ap.R < ap.rank;
    for (int r = 0; r < ap.R; ++r) { ap.inv[r] = sm.S(r, r); if (ap.inv[r] != 1) ap.masked = true; }

    // The columns of V are not unique: a kernel column may be added to any other column
    // without changing S = U A V.  If no column moves the output index alpha by exactly one
    // element of df, use that freedom on ONE column to obtain such a direction (consecutive
    // values of that loop variable then read df contiguously).  Kernel columns are oriented
    // so that df is walked forward.
    {
        const int kap = ap.kappa, R = ap.R;
        std::vector<int64_t> fstride(ap.n, 0);           // flat stride of df per column (0 for sum indices)
        int64_t st = 1;
        for (int d = p.n_out - 1; d >= 0; --d) { fstride[d] = st; st = mul_ck(st, p.out_shape[d]); }
        auto df_stride = [&](const std::vector<int64_t> &col) {
            int64_t s = 0;
            for (int d = 0; d < ap.n; ++d) s = add_ck(s, mul_ck(fstride[d], col[d]));
            return s;
        };
        auto column = [&](int c) { std::vector<int64_t> v(ap.n); for (int d = 0; d < ap.n; ++d) v[d] = ap.V(d, c); return v; };
        bool have_contiguous = false;
        for (int c = 0; c < ap.n; ++c) if (std::llabs(df_stride(column(c))) == 1) have_contiguous = true;
        int best_col = -1; int64_t best_mag = 0;
        std::vector<int64_t> best_vec;
        for (int c = 0; c < ap.n && !have_contiguous && kap > 0; ++c) {
            std::vector<int> coef(kap, -2);
            for (;;) {
                std::vector<int64_t> cand = column(c);
                bool skip = false;
                for (int m = 0; m < kap; ++m) {
                    if (R + m == c) { if (coef[m] != 0) skip = true; continue; }
                    for (int d = 0; d < ap.n; ++d) cand[d] = add_ck(cand[d], mul_ck(coef[m], ap.V(d, R + m)));
                }
                if (!skip && std::llabs(df_stride(cand)) == 1) {
                    int64_t mag = 0;
                    for (int64_t v : cand) mag += std::llabs(v);
                    if (best_col < 0 || mag < best_mag) { best_col = c; best_mag = mag; best_vec = cand; }
                }
                int m = 0;
                while (m < kap && ++coef[m] > 2) { coef[m] = -2; ++m; }
                if (m == kap) break;
            }
        }
        if (best_col >= 0) for (int d = 0; d < ap.n; ++d) ap.V(d, best_col) = best_vec[d];
        for (int m = 0; m < kap; ++m) {
            int64_t s = df_stride(column(R + m));
            bool flip = s < 0;
            if (s == 0) for (int d = 0; d < ap.n; ++d) if (ap.V(d, R + m) != 0) { flip = ap.V(d, R + m) < 0; break; }
            if (flip) for (int d = 0; d < ap.n; ++d) ap.V(d, R + m) = neg_ck(ap.V(d, R + m));
        }
    }
    ap.Vinv = unimodular_inverse(ap.V);
    ap.zorder.resize(ap.kappa);
    for (int l = 0; l < ap.kappa; ++l) ap.zorder[l] = l;
    compute_bounds(ap);
    // bounding box of x' = (V^-1 alpha_hat)_{1..R} over the index box
    ap.xlo.resize(ap.R); ap.xhi.resize(ap.R);
    for (int j = 0; j < ap.R; ++j) {
        std::vector<int64_t> c(ap.n);
        for (int d = 0; d < ap.n; ++d) c[d] = ap.Vinv(j, d);
        affine_range(0, c, ap.box_lo, ap.box_hi, ap.xlo[j], ap.xhi[j]);
    }
}

namespace {

struct EnumCtx {
    const AccessPlan *ap;
    std::vector<int64_t> x, z;
    std::vector<int64_t> *out;
    size_t cap, count;
};

int64_t row_num(const BoundRowH &r, const std::vector<int64_t> &x, const std::vector<int64_t> &z)
{
    int64_t v = r.c0;
    for (size_t j = 0; j < r.cx.size(); ++j) v = add_ck(v, mul_ck(r.cx[j], x[j]));
    for (size_t m = 0; m < r.cz.size(); ++m) if (r.cz[m]) v = add_ck(v, mul_ck(r.cz[m], z[m]));
    return v;
}

void enum_level(EnumCtx &c, int l)
{
    const AccessPlan &ap = *c.ap;
    if (l == ap.kappa) {
        if (c.out && c.count < c.cap)
            for (int d = 0; d < ap.n; ++d) {
                int64_t v = 0;
                for (int j = 0; j < ap.R; ++j) v = add_ck(v, mul_ck(ap.V(d, j), c.x[j]));
                for (int m = 0; m < ap.kappa; ++m) v = add_ck(v, mul_ck(ap.V(d, ap.R + ap.zorder[m]), c.z[m]));
                c.out->push_back(v);
            }
        ++c.count;
        return;
    }
    int64_t lo = INT64_MIN, hi = INT64_MAX;
    for (const BoundRowH &r : ap.lower[l]) lo = std::max(lo, ceil_div(row_num(r, c.x, c.z), r.den));
    for (const BoundRowH &r : ap.upper[l]) hi = std::min(hi, floor_div(row_num(r, c.x, c.z), r.den));
    for (int64_t v = lo; v <= hi; ++v) { c.z[l] = v; enum_level(c, l + 1); }
    c.z[l] = 0;
}

}  // namespace

size_t enumerate_access(const tad_plan &p, int q, const int64_t *beta, std::vector<int64_t> *out, size_t cap)
{
    const AccessPlan &ap = p.access[q];
    // b' = U (beta - o); cokernel rows must vanish, invariant factors must divide (Sec. 4.1)
    std::vector<int64_t> bp(ap.rank, 0);
    for (int r = 0; r < ap.rank; ++r)
        for (int c = 0; c < ap.rank; ++c) bp[r] = add_ck(bp[r], mul_ck(ap.U(r, c), sub_ck(beta[c], ap.off[c])));
    for (int r = ap.R; r < ap.rank; ++r) if (bp[r] != 0) return 0;
    EnumCtx c;
    c.ap = &ap; c.out = out; c.cap = cap; c.count = 0;
    c.x.resize(ap.R); c.z.assign(ap.kappa, 0);
    for (int r = 0; r < ap.R; ++r) {
        if (bp[r] % ap.inv[r] != 0) return 0;
        c.x[r] = bp[r] / ap.inv[r];
    }
    for (const BoundRowH &g : ap.guards) if (row_num(g, c.x, c.z) > 0) return 0;
    enum_level(c, 0);
    return c.count;
}

}  // namespace tad

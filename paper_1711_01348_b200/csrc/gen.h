// Derivative-graph instances (host only): the values a kernel computes, as a DAG over the kernel's
// loop variables, built by scalar reverse-mode differentiation (Sec. 2) with the sums on the path
// to the leaf liberated (Sec. 5.2).  Shared by the bytecode emitter and the contraction planner.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <tuple>

#include "plan.h"

namespace tad {

// ---- derivative-graph instances -------------------------------------------------------
enum IOp {
    I_CONST, I_LOAD, I_NEG, I_EXP, I_LOG, I_SIN, I_COS, I_TANH, I_SINH, I_COSH,
    I_SQR, I_POWI, I_ADD, I_SUB, I_MUL, I_DIV, I_MULC, I_ADDC, I_SUM
};

struct Inst {
    int op = I_CONST, a = -1, b = -1;
    int load = -1;          // I_LOAD
    int ipow = 0;           // I_POWI
    float imm = 0.f;        // I_CONST, I_MULC, I_ADDC
    int var = -1;           // I_SUM: bound loop variable
    int64_t lo = 0, hi = -1;// I_SUM
    uint32_t deps = 0;      // kernel variables it depends on
    uint32_t adeps = 0;     // alpha_hat positions (free) it depends on; bit 16+v for bound variable v
    int uses = 0;
    int temp = -1;
    int home_sum = -1;      // innermost bound-sum instance whose variable it depends on (-1: none)
    int zlevel = 0;         // 1 + deepest kernel-coordinate loop it depends on, 0 if none
};

struct VarInfo {
    int kind;               // 0 outer, 1 kernel coordinate, 2 bound sum
    int64_t ext;            // extent (exact for outer and bound sums, estimate for kernel coordinates)
    int sum_inst;           // kind 2
};

struct Gen {
    tad_plan &p;
    int q;                               // index expression being differentiated, -1 for forward
    int n_outer = 0, kappa = 0;
    std::vector<VarInfo> vars;
    // affine map of every alpha_hat position over (outer, kernel-coordinate) variables
    std::vector<int64_t> a_c0;
    std::vector<std::vector<int64_t>> a_coef;
    std::vector<bool> a_free_ok;
    std::vector<Inst> inst;
    std::map<std::tuple<int, int, int, int, int, int32_t, int>, int> cse;
    std::vector<TadpLoad> loads;
    std::map<std::pair<int, uint32_t>, int> val_memo;        // (node, free set) -> inst
    std::map<std::pair<int, uint32_t>, int> bound_var;       // (sum slot, free set) -> var
    std::vector<int> zorder;                                  // loop l -> kernel column
    std::vector<int> zpos;                                    // kernel column -> loop position
    int lane_var = -1;
    int unroll_var = -1;                                      // element variable B (-1: none)
    std::map<int, int> staged;                                // sum node -> pointer slot of its staged adjoint
    std::vector<int> stages_used;                             // pointer slots the derivative reads
    bool use_f = false;                                       // the value of the root is read from the saved forward output
    bool reads_f = false;

    Gen(tad_plan &pl, int acc) : p(pl), q(acc) {}

    int n_idx() const { return p.n_out + p.n_sum; }

    // -- instance construction with common-subexpression elimination
    int intern(Inst in)
    {
        int32_t immbits; std::memcpy(&immbits, &in.imm, 4);
        auto key = std::make_tuple(in.op, in.a, in.b, in.load, in.ipow, immbits, in.var);
        auto it = cse.find(key);
        if (it != cse.end()) return it->second;
        if (in.op != I_CONST && in.op != I_LOAD && in.op != I_SUM) {
            in.deps = inst[in.a].deps | (in.b >= 0 ? inst[in.b].deps : 0);
            in.adeps = inst[in.a].adeps | (in.b >= 0 ? inst[in.b].adeps : 0);
        }
        inst.push_back(in);
        cse[key] = (int)inst.size() - 1;
        return (int)inst.size() - 1;
    }
    int konst(float v) { Inst i; i.op = I_CONST; i.imm = v; return intern(i); }
    int un(int op, int a) { Inst i; i.op = op; i.a = a; return intern(i); }
    int neg(int a) { if (inst[a].op == I_NEG) return inst[a].a; return un(I_NEG, a); }
    int mulc(int a, float c)
    {
        if (c == 1.f) return a;
        if (inst[a].op == I_CONST) return konst(inst[a].imm * c);
        Inst i; i.op = I_MULC; i.a = a; i.imm = c; return intern(i);
    }
    int addc(int a, float c)
    {
        if (c == 0.f) return a;
        if (inst[a].op == I_CONST) return konst(inst[a].imm + c);
        Inst i; i.op = I_ADDC; i.a = a; i.imm = c; return intern(i);
    }
    int bin(int op, int a, int b)
    {
        if (op == I_MUL) {
            if (inst[a].op == I_CONST) return mulc(b, inst[a].imm);
            if (inst[b].op == I_CONST) return mulc(a, inst[b].imm);
            if (a == b) return un(I_SQR, a);
            if (a > b) std::swap(a, b);
        }
        if (op == I_ADD) {
            if (inst[a].op == I_CONST) return addc(b, inst[a].imm);
            if (inst[b].op == I_CONST) return addc(a, inst[b].imm);
            if (a > b) std::swap(a, b);
        }
        if (op == I_SUB && inst[b].op == I_CONST) return addc(a, -inst[b].imm);
        if (op == I_DIV && inst[b].op == I_CONST) return mulc(a, 1.f / inst[b].imm);
        Inst i; i.op = op; i.a = a; i.b = b; return intern(i);
    }
    int powi(int a, int n)
    {
        if (n == 0) return konst(1.f);
        if (n == 1) return a;
        if (n == 2) return un(I_SQR, a);
        Inst i; i.op = I_POWI; i.a = a; i.ipow = n; return intern(i);
    }

    // -- loads: element offset affine in the kernel variables
    int make_load(int ptr, const std::vector<int64_t> &A, const std::vector<int64_t> &off, int rank,
                  const std::vector<int64_t> &shape, uint32_t free_set, uint32_t scope)
    {
        std::vector<int64_t> stride(rank, 1);
        for (int r = rank - 2; r >= 0; --r) stride[r] = mul_ck(stride[r + 1], shape[r + 1]);
        int64_t base = 0, elems = 1;
        for (int r = 0; r < rank; ++r) { base = add_ck(base, mul_ck(stride[r], off[r])); elems *= shape[r]; }
        std::vector<int64_t> coef(TADP_MAX_VARS, 0);
        uint32_t adeps = 0;
        const int nidx = n_idx();
        for (int d = 0; d < nidx; ++d) {
            int64_t flat = 0;
            for (int r = 0; r < rank; ++r) flat = add_ck(flat, mul_ck(stride[r], A[size_t(r) * nidx + d]));
            if (flat == 0) continue;
            bool is_sum = d >= p.n_out;
            int s = d - p.n_out;
            if (is_sum && !(free_set & (1u << s))) {
                if (!(scope & (1u << s))) throw BadExpr("internal: load reads a sum index outside its sum");
                auto it = bound_var.find({s, free_set});
                if (it == bound_var.end()) throw BadExpr("internal: bound sum variable missing");
                coef[it->second] = add_ck(coef[it->second], flat);
                adeps |= 1u << (16 + it->second);
            } else {
                if (!a_free_ok[d]) throw BadExpr("internal: free index without an affine map");
                base = add_ck(base, mul_ck(flat, a_c0[d]));
                for (size_t v = 0; v < a_coef[d].size(); ++v)
                    coef[v] = add_ck(coef[v], mul_ck(flat, a_coef[d][v]));
                adeps |= 1u << d;
            }
        }
        TadpLoad L{};
        L.ptr = ptr;
        if (std::llabs(base) >= (int64_t(1) << 31)) throw Overflow();
        L.base = (int32_t)base;
        uint32_t deps = 0;
        for (int v = 0; v < TADP_MAX_VARS; ++v) {
            if (std::llabs(coef[v]) >= (int64_t(1) << 31)) throw Overflow();
            L.coef[v] = (int32_t)coef[v];
            if (coef[v]) deps |= 1u << v;
        }
        L.limit = (int32_t)elems;
        int id = -1;
        for (size_t i = 0; i < loads.size(); ++i)
            if (!std::memcmp(&loads[i], &L, sizeof L)) id = (int)i;
        if (id < 0) {
            if ((int)loads.size() >= TADP_MAX_LOADS) throw Unsupported("too many distinct loads in one kernel");
            loads.push_back(L); id = (int)loads.size() - 1;
        }
        Inst in; in.op = I_LOAD; in.load = id; in.deps = deps; in.adeps = adeps;
        return intern(in);
    }

    int new_var(int kind, int64_t ext)
    {
        if ((int)vars.size() >= TADP_MAX_VARS) throw Unsupported("too many loop variables in one kernel");
        vars.push_back({kind, ext, -1});
        return (int)vars.size() - 1;
    }

    // -- value of an expression node with the sums of `free_set` liberated (taken from alpha_hat)
    int val(int n, uint32_t free_set)
    {
        const NodeH &nd = p.nodes[n];
        if (nd.op == TAD_OP_CONST) return konst((float)nd.imm);
        if (use_f && n == (int)p.nodes.size() - 1 && free_set == 0) {
            // f[alpha] as the forward pass wrote it
            std::vector<int64_t> A(size_t(p.n_out) * n_idx(), 0), off(p.n_out, 0);
            for (int d = 0; d < p.n_out; ++d) A[size_t(d) * n_idx() + d] = 1;
            reads_f = true;
            return make_load(TADP_F_SLOT, A, off, p.n_out, p.out_shape, 0, 0);
        }
        auto key = std::make_pair(n, free_set);
        auto it = val_memo.find(key);
        if (it != val_memo.end()) return it->second;
        int r = -1;
        switch (nd.op) {
        case TAD_OP_LOAD: {
            int arg = p.accArg[nd.access];
            r = make_load(arg, p.accA[nd.access], p.accOff[nd.access], (int)p.arg_shape[arg].size(),
                          p.arg_shape[arg], free_set, nd.scope);
            break;
        }
        case TAD_OP_NEG: r = neg(val(nd.in0, free_set)); break;
        case TAD_OP_ADD: { int a = val(nd.in0, free_set), b = val(nd.in1, free_set); r = bin(I_ADD, a, b); break; }
        case TAD_OP_SUB: { int a = val(nd.in0, free_set), b = val(nd.in1, free_set); r = bin(I_SUB, a, b); break; }
        case TAD_OP_MUL: { int a = val(nd.in0, free_set), b = val(nd.in1, free_set); r = bin(I_MUL, a, b); break; }
        case TAD_OP_DIV: { int a = val(nd.in0, free_set), b = val(nd.in1, free_set); r = bin(I_DIV, a, b); break; }
        case TAD_OP_POWI: r = powi(val(nd.in0, free_set), nd.ipow); break;
        case TAD_OP_EXP: r = un(I_EXP, val(nd.in0, free_set)); break;
        case TAD_OP_LOG: r = un(I_LOG, val(nd.in0, free_set)); break;
        case TAD_OP_SIN: r = un(I_SIN, val(nd.in0, free_set)); break;
        case TAD_OP_COS: r = un(I_COS, val(nd.in0, free_set)); break;
        case TAD_OP_TANH: r = un(I_TANH, val(nd.in0, free_set)); break;
        case TAD_OP_SINH: r = un(I_SINH, val(nd.in0, free_set)); break;
        case TAD_OP_COSH: r = un(I_COSH, val(nd.in0, free_set)); break;
        case TAD_OP_SUM: {
            int s = nd.sum_idx - p.n_out;
            int v = new_var(2, nd.sum_hi - nd.sum_lo + 1);
            bound_var[{s, free_set}] = v;
            int body = val(nd.in0, free_set);
            Inst in; in.op = I_SUM; in.a = body; in.var = v; in.lo = nd.sum_lo; in.hi = nd.sum_hi;
            in.deps = inst[body].deps & ~(1u << v);
            in.adeps = inst[body].adeps & ~(1u << (16 + v));
            r = intern(in);
            vars[v].sum_inst = r;
            break;
        }
        default: throw BadExpr("unknown operation");
        }
        val_memo[key] = r;
        return r;
    }

    // -- reverse accumulation (Sec. 2): the adjoint of the root is df; returns the term Delta
    //    of Sec. 5.3, i.e. df * d f / d x^{pq} with every sum on the path to the leaf liberated
    //    With target >= 0 the accumulation stops at that node and its adjoint is returned.
    int differentiate(int df_inst, int target = -1)
    {
        const int root = (int)p.nodes.size() - 1;
        std::vector<bool> active(p.nodes.size(), false);
        for (int n = 0; n <= root; ++n) {
            const NodeH &nd = p.nodes[n];
            if (!nd.reachable) continue;
            if (target >= 0) { if (n == target) { active[n] = true; continue; } }
            else if (nd.op == TAD_OP_LOAD) { active[n] = nd.access == q; continue; }
            active[n] = (nd.in0 >= 0 && active[nd.in0]) || (nd.in1 >= 0 && active[nd.in1]);
        }
        // need[n]: the adjoint of n has to be built from its consumers (it is not staged and
        // some path from it reaches a wanted leaf without crossing a staged node first)
        std::vector<bool> need(p.nodes.size(), false);
        for (int n = 0; n <= root; ++n) {
            if (!active[n]) continue;
            const NodeH &nd = p.nodes[n];
            bool leaf = target >= 0 ? n == target : (nd.op == TAD_OP_LOAD && nd.access == q);
            bool below = false;
            for (int c : {nd.in0, nd.in1})
                if (c >= 0 && active[c] && need[c]) below = true;
            need[n] = !staged.count(n) && (leaf || below);
        }
        std::vector<int> adj(p.nodes.size(), -1);
        if (!active[root]) return -1;
        adj[root] = df_inst;
        int total = -1;
        auto wants = [&](int c) { return c >= 0 && active[c] && need[c]; };
        auto push = [&](int c, int x) { adj[c] = adj[c] < 0 ? x : bin(I_ADD, adj[c], x); };
        for (int n = root; n >= 0; --n) {
            if (!active[n]) continue;
            const NodeH &nd = p.nodes[n];
            const uint32_t F = nd.scope;          // every enclosing sum lies on the path: liberated
            int g = adj[n];
            auto st = staged.find(n);
            if (st != staged.end()) {
                // the adjoint of this sum was evaluated once per alpha by a staging kernel
                std::vector<int64_t> A(size_t(p.n_out) * n_idx(), 0), off(p.n_out, 0);
                for (int d = 0; d < p.n_out; ++d) A[size_t(d) * n_idx() + d] = 1;
                g = make_load(st->second, A, off, p.n_out, p.out_shape, F, F);
                if (std::find(stages_used.begin(), stages_used.end(), st->second) == stages_used.end())
                    stages_used.push_back(st->second);
            }
            if (g < 0) continue;
            if (n == target) return g;
            const int a = nd.in0, b = nd.in1;
            switch (nd.op) {
            case TAD_OP_LOAD: if (nd.access == q && target < 0) total = total < 0 ? g : bin(I_ADD, total, g); break;
            case TAD_OP_NEG: if (wants(a)) push(a, neg(g)); break;
            case TAD_OP_ADD: if (wants(a)) push(a, g); if (wants(b)) push(b, g); break;
            case TAD_OP_SUB: if (wants(a)) push(a, g); if (wants(b)) push(b, neg(g)); break;
            case TAD_OP_MUL:
                if (wants(a)) push(a, bin(I_MUL, g, val(b, F)));
                if (wants(b)) push(b, bin(I_MUL, g, val(a, F)));
                break;
            case TAD_OP_DIV:
                if (wants(a)) push(a, bin(I_DIV, g, val(b, F)));
                if (wants(b)) push(b, neg(bin(I_DIV, bin(I_MUL, g, val(n, F)), val(b, F))));
                break;
            case TAD_OP_POWI:
                if (nd.ipow != 0 && wants(a))
                    push(a, bin(I_MUL, g, mulc(powi(val(a, F), nd.ipow - 1), (float)nd.ipow)));
                break;
            case TAD_OP_EXP: if (wants(a)) push(a, bin(I_MUL, g, val(n, F))); break;
            case TAD_OP_LOG: if (wants(a)) push(a, bin(I_DIV, g, val(a, F))); break;
            case TAD_OP_SIN: if (wants(a)) push(a, bin(I_MUL, g, un(I_COS, val(a, F)))); break;
            case TAD_OP_COS: if (wants(a)) push(a, neg(bin(I_MUL, g, un(I_SIN, val(a, F))))); break;
            case TAD_OP_TANH:
                if (wants(a)) { int t = val(n, F); push(a, bin(I_MUL, g, addc(neg(un(I_SQR, t)), 1.f))); }
                break;
            case TAD_OP_SINH: if (wants(a)) push(a, bin(I_MUL, g, un(I_COSH, val(a, F)))); break;
            case TAD_OP_COSH: if (wants(a)) push(a, bin(I_MUL, g, un(I_SINH, val(a, F)))); break;
            case TAD_OP_SUM: if (wants(a)) push(a, g); break;     // d s-bar / d s = 1 at the liberated index
            default: break;
            }
        }
        return total;
    }
};

inline int32_t to_i32(int64_t v) { if (std::llabs(v) >= (int64_t(1) << 31)) throw Overflow(); return (int32_t)v; }

// ---- affine description of a contraction (contract_gen.cpp) ---------------------------------
struct AVar { int64_t ext; bool reduce; };               // values 0 .. ext-1 after normalisation
struct AMap { int ptr = 0; int64_t base = 0, limit = 0; std::vector<int64_t> coef; };   // limit: elements in the tensor
struct AGuard { std::vector<int64_t> coef; int64_t c0 = 0, ext = 1; };   // live iff 0 <= c0 + coef . vars < ext

struct System {
    std::vector<AVar> vars;
    AMap A, B, O;
    std::vector<AGuard> guards;
    bool loose_box = false;     // the outer box is a bounding box of the live elements, not the set itself
};

// builds one contraction program from a system whose loops all have fixed ranges; an operand with ptr < 0 is
// a tensor of ones (a plain summation of the other operand).  strict_fill: refuse mostly empty tiles
bool emit_program(const System &s, float scale, int accumulate, bool allow_split, bool strict_fill, TadcProgram &P, std::string &text);

// contract_gen.cpp: recognises a kernel whose term is a product of two index expressions summed over
// loops with fixed ranges and fills k.contract; returns false (and leaves k alone) otherwise.
// allow_split: the caller has a workspace for partial sums of a split summation
bool try_contraction(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
                     const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards);

// line_gen.cpp: a gradient kernel whose term is a product of index expressions becomes a line-sum program
bool try_line(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
              const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards);
// factor.cpp: the expression optimisation pass; fills k.pre / k.aux and emits the kernel itself when it
// finds summations worth pushing inside the term, returns false (k untouched) otherwise
bool try_factoring(Gen &g, Kernel &k, int root, int scale, bool allow_split, const std::vector<std::vector<TadpRow>> &lower,
                   const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards);
// codegen.cpp: schedules and emits one kernel without running the optimisation pass on it
void emit_plain_kernel(Gen &g, Kernel &k, int root, const std::vector<std::vector<TadpRow>> &lower,
                       const std::vector<std::vector<TadpRow>> &upper, const std::vector<TadpRow> &guards, bool allow_split);

}  // namespace tad

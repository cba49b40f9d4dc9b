// Host-side plan: validated expression, per-index-expression integer analysis (Smith normal
// form, kernel / cokernel, Fourier-Motzkin bound rows) and the compiled device programs.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "../../include/tad.h"
#include "intalg.h"
#include "program.h"
#include "contract.h"
#include "ew.h"
#include "line.h"

namespace tad {

struct BadExpr : std::runtime_error { explicit BadExpr(const std::string &m) : std::runtime_error(m) {} };
struct OutOfRange : std::runtime_error { explicit OutOfRange(const std::string &m) : std::runtime_error(m) {} };
struct InvalidArg : std::runtime_error { explicit InvalidArg(const std::string &m) : std::runtime_error(m) {} };

struct NodeH {
    int op, in0, in1, access, ipow, sum_idx;
    int64_t sum_lo, sum_hi;
    double imm;
    uint32_t scope = 0;        // bit s set: enclosed by the sum whose index is alpha_hat[n_out + s]
    bool reachable = false;
};

// A bound row in host form: value = (c0 + sum_j cx[j] x'_j + sum_m cz[m] z_m) / den.
struct BoundRowH {
    int64_t den = 1, c0 = 0;
    std::vector<int64_t> cx;   // R entries (over x')
    std::vector<int64_t> cz;   // kappa entries (over z in loop order, only outer loops non-zero)
};

struct AccessPlan {
    int arg = 0, rank = 0;
    int n = 0;                         // columns of A-hat
    std::vector<int> idx_pos;          // alpha_hat position of every column
    uint32_t scope = 0;                // enclosing sums
    bool used = false;                 // some reachable load node reads through it
    Mat A;                             // rank x n (restricted to idx_pos)
    std::vector<int64_t> off;          // rank
    std::vector<int64_t> box_lo, box_hi;   // per column, inclusive
    // Smith normal form S = U A V
    Mat U, V, Vinv;
    std::vector<int64_t> inv;          // invariant factors alpha_1..alpha_R
    int R = 0, kappa = 0;
    bool masked = false;               // cokernel rows exist or some invariant factor > 1
    std::vector<int> zorder;           // loop l (0 = outermost) iterates kernel column V[:, R + zorder[l]]
    // bound rows per loop (in loop order), guards (rows over x' only that must be <= 0)
    std::vector<std::vector<BoundRowH>> lower, upper;
    std::vector<BoundRowH> guards;
    // x' bounding box (inclusive) over which the live elements lie
    std::vector<int64_t> xlo, xhi;
    int lane_var = -1;                 // filled by the code generator (index into kernel variables)
};

struct KernelStats {
    int64_t outputs = 0, terms = 0;
    double alg_bytes = 0, alg_flops = 0, alg_trans = 0;
    int bytecode_words = 0, n_launches = 0;
};

struct Kernel {
    TadpProgram prog;
    int out_arg = -1;          // -1: forward (writes f); else the argument whose gradient it writes
    int access = -1;
    int vec = 4;               // elements per thread along the lane variable (TA)
    int vec_u = 1;             // elements per thread along the element variable (UB)
    bool rich = false;         // the build of the shape with more registers per thread and fewer warps per SM
    std::vector<int> stages_used;   // backward: staged adjoints it reads (indices into tad_plan::stages)
    std::vector<TadcProgram> contract;   // non-empty: the kernel is a contraction, run by the tile kernel (one launch per
                                         // program) instead of the interpreter
    std::vector<TadeProgram> ew;         // non-empty: a kernel without loops, run by the element-wise kernel
    std::vector<TadlProgram> line;       // non-empty: sums of products of index expressions, run by the line-sum kernel
    // Expression optimisation: tensors in the auxiliary area of the workspace and the kernels that fill them
    // (launched in this order before the kernel itself, each writing the tensor out_aux)
    struct Aux { size_t offset = 0, bytes = 0; int slot = 0; };
    std::vector<Aux> aux;
    size_t aux_bytes = 0;
    std::vector<Kernel> pre;
    int out_aux = -1;
    KernelStats stats;
    std::string listing;
};

}  // namespace tad

struct tad_plan {
    // expression
    int n_out = 0, n_sum = 0, n_args = 0;
    std::vector<int64_t> out_shape;
    std::vector<std::vector<int64_t>> arg_shape;
    std::vector<int64_t> arg_elems;
    int64_t out_elems = 0;
    std::vector<tad::NodeH> nodes;
    std::vector<int64_t> sum_lo, sum_hi;       // per sum index
    std::vector<int> sum_node;                 // node id of the sum that owns each sum index
    std::vector<std::vector<int64_t>> accA;    // raw access matrices (rank x n_idx) and offsets
    std::vector<std::vector<int64_t>> accOff;
    std::vector<int> accArg;
    tad_options opt{};
    // analysis + programs
    std::vector<tad::AccessPlan> access;
    tad::Kernel forward;
    std::vector<tad::Kernel> stages;            // staged adjoints of top-level sums, one |f|-sized buffer each
    std::vector<int> stage_node;                // the sum node each stage belongs to
    std::vector<tad::Kernel> backward;          // one per used index expression
    std::vector<std::vector<int>> arg_kernels;  // per argument: indices into backward, launch order
    std::vector<bool> arg_zero_fill;            // the gradient is cleared before its kernels add into it
    size_t partial_bytes = 0;                   // workspace for the partial sums of split summations (largest kernel)
    size_t aux_bytes = 0;                       // workspace for auxiliary tensors (largest kernel)
    mutable void *side = nullptr;               // second stream and its events (independent memory-bound passes run beside a contraction)
    mutable void *host_step = nullptr;          // streams and events of tad_step_host, created by its first call
};

// runtime.cu: releases what tad_step_host created for this plan (tad_destroy calls it)
void tad_release_host_step(const tad_plan *plan);

namespace tad {

// plan.cpp
void build_expression(tad_plan &p, const tad_expr *e, const tad_options *opt);
void analyse_access(tad_plan &p, int q);
void compute_bounds(AccessPlan &ap);   // recompute bound rows after ap.zorder changed
// Enumerates Gamma-hat(beta) by walking the plan; appends alpha_hat vectors (n each) to out (if non-null).
size_t enumerate_access(const tad_plan &p, int q, const int64_t *beta, std::vector<int64_t> *out, size_t cap);

// codegen.cpp
void generate_forward(tad_plan &p);
void generate_stages(tad_plan &p);
void generate_backward(tad_plan &p, int q);

// print.cpp: the expression (which = -1) or the derivative through index expression `which` in the notation of Sec. 6
std::string print_expression(const tad_plan &p, int which, const char *const *arg_names, const char *const *idx_names);

}  // namespace tad

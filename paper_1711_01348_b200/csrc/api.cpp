// C ABI, host-only part: compile, introspection and the exported pieces of the integer algebra.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>

#include "plan.h"

namespace tad {
thread_local std::string g_last_error;
void set_error(const std::string &m) { g_last_error = m; }

template <class F> tad_status guarded(F &&f)
{
    try { f(); return TAD_OK; }
    catch (const InvalidArg &e) { set_error(e.what()); return TAD_ERR_INVALID_ARG; }
    catch (const BadExpr &e) { set_error(e.what()); return TAD_ERR_BAD_EXPR; }
    catch (const OutOfRange &e) { set_error(e.what()); return TAD_ERR_OUT_OF_RANGE; }
    catch (const Overflow &e) { set_error(e.what()); return TAD_ERR_OVERFLOW; }
    catch (const Unsupported &e) { set_error(e.what()); return TAD_ERR_UNSUPPORTED; }
    catch (const std::bad_alloc &) { set_error("out of host memory"); return TAD_ERR_NOMEM; }
    catch (const std::exception &e) { set_error(e.what()); return TAD_ERR_INVALID_ARG; }
}
}  // namespace tad

using namespace tad;

extern "C" {

const char *tad_last_error(void) { return g_last_error.c_str(); }

tad_status tad_compile(const tad_expr *expr, const tad_options *opt, tad_plan **out)
{
    if (!out) { set_error("out is NULL"); return TAD_ERR_INVALID_ARG; }
    tad_plan *p = nullptr;
    tad_status st = guarded([&] {
        p = new tad_plan();
        build_expression(*p, expr, opt);
        for (int q = 0; q < (int)p->access.size(); ++q)
            if (p->access[q].used) analyse_access(*p, q);
        generate_forward(*p);
        generate_stages(*p);
        p->arg_kernels.assign(p->n_args, {});
        p->arg_zero_fill.assign(p->n_args, false);
        for (int q = 0; q < (int)p->access.size(); ++q)
            if (p->access[q].used && p->access[q].masked) p->arg_zero_fill[p->access[q].arg] = true;
        p->backward.reserve(p->access.size());
        for (int q = 0; q < (int)p->access.size(); ++q)
            if (p->access[q].used) generate_backward(*p, q);
    });
    if (st != TAD_OK) { delete p; return st; }
    *out = p;
    return TAD_OK;
}

void tad_destroy(tad_plan *plan) { if (plan) tad_release_host_step(plan); delete plan; }

int32_t tad_plan_num_stages(const tad_plan *plan) { return plan ? (int32_t)plan->stages.size() : 0; }

tad_status tad_plan_access_info(const tad_plan *plan, int32_t access, tad_access_info *out)
{
    return guarded([&] {
        if (!plan || !out) throw InvalidArg("NULL argument");
        if (access < 0 || access >= (int)plan->access.size() || !plan->access[access].used)
            throw InvalidArg("no such index expression (or it is never read)");
        const AccessPlan &ap = plan->access[access];
        std::memset(out, 0, sizeof *out);
        out->arg = ap.arg; out->rank = ap.rank; out->n_idx = ap.n; out->R = ap.R; out->kappa = ap.kappa;
        out->masked = ap.masked; out->lane_var = ap.lane_var;
        for (int c = 0; c < ap.n; ++c) { out->idx_pos[c] = ap.idx_pos[c]; out->box_lo[c] = ap.box_lo[c]; out->box_hi[c] = ap.box_hi[c]; }
        for (int r = 0; r < ap.rank; ++r) {
            out->offset[r] = ap.off[r];
            for (int c = 0; c < ap.n; ++c) out->A[r * ap.n + c] = ap.A(r, c);
            for (int c = 0; c < ap.rank; ++c) out->U[r * ap.rank + c] = ap.U(r, c);
        }
        for (int r = 0; r < ap.R; ++r) out->S[r] = ap.inv[r];
        // V with its kernel columns in loop order
        for (int r = 0; r < ap.n; ++r) {
            for (int c = 0; c < ap.R; ++c) out->V[r * ap.n + c] = ap.V(r, c);
            for (int l = 0; l < ap.kappa; ++l) out->V[r * ap.n + ap.R + l] = ap.V(r, ap.R + ap.zorder[l]);
        }
        for (int l = 0; l < ap.kappa; ++l) { out->n_lower[l] = (int)ap.lower[l].size(); out->n_upper[l] = (int)ap.upper[l].size(); }
    });
}

tad_status tad_plan_bound_row(const tad_plan *plan, int32_t access, int32_t loop, int32_t upper,
                              int32_t row, int64_t *den, int64_t *c0, int64_t *coef_x, int64_t *coef_z)
{
    return guarded([&] {
        if (!plan || !den || !c0) throw InvalidArg("NULL argument");
        if (access < 0 || access >= (int)plan->access.size() || !plan->access[access].used) throw InvalidArg("no such index expression");
        const AccessPlan &ap = plan->access[access];
        if (loop < 0 || loop >= ap.kappa) throw InvalidArg("no such loop");
        const auto &rows = upper ? ap.upper[loop] : ap.lower[loop];
        if (row < 0 || row >= (int)rows.size()) throw InvalidArg("no such row");
        *den = rows[row].den; *c0 = rows[row].c0;
        if (coef_x) for (int j = 0; j < ap.R; ++j) coef_x[j] = rows[row].cx[j];
        if (coef_z) for (int m = 0; m < loop; ++m) coef_z[m] = rows[row].cz[m];
    });
}

tad_status tad_plan_enumerate(const tad_plan *plan, int32_t access, const int64_t *beta,
                              int64_t *alpha_hat_out, size_t cap, size_t *n_terms)
{
    return guarded([&] {
        if (!plan || !beta || !n_terms) throw InvalidArg("NULL argument");
        if (access < 0 || access >= (int)plan->access.size() || !plan->access[access].used) throw InvalidArg("no such index expression");
        std::vector<int64_t> buf;
        size_t n = enumerate_access(*plan, access, beta, alpha_hat_out ? &buf : nullptr, cap);
        if (alpha_hat_out && !buf.empty()) std::memcpy(alpha_hat_out, buf.data(), buf.size() * sizeof(int64_t));
        *n_terms = n;
    });
}

static const Kernel *pick_kernel(const tad_plan *plan, int32_t which)
{
    if (which == -1) return &plan->forward;
    if (which <= -2 && -2 - which < (int)plan->stages.size()) return &plan->stages[-2 - which];
    for (const Kernel &k : plan->backward) if (k.access == which) return &k;
    return nullptr;
}

tad_status tad_plan_kernel_stats(const tad_plan *plan, int32_t which, tad_kernel_stats *out)
{
    return guarded([&] {
        if (!plan || !out) throw InvalidArg("NULL argument");
        const Kernel *k = pick_kernel(plan, which);
        if (!k) throw InvalidArg("no such kernel");
        out->outputs = k->stats.outputs; out->terms = k->stats.terms;
        out->alg_bytes = k->stats.alg_bytes; out->alg_flops = k->stats.alg_flops;
        out->alg_transcendentals = k->stats.alg_trans;
        out->bytecode_words = k->stats.bytecode_words; out->n_launches = k->stats.n_launches;
    });
}

size_t tad_plan_disassemble(const tad_plan *plan, int32_t which, char *buf, size_t cap)
{
    if (!plan) return 0;
    const Kernel *k = pick_kernel(plan, which);
    if (!k) return 0;
    if (buf && cap) {
        size_t n = std::min(cap - 1, k->listing.size());
        std::memcpy(buf, k->listing.data(), n);
        buf[n] = 0;
    }
    return k->listing.size() + 1;
}

size_t tad_plan_print(const tad_plan *plan, int32_t which, const char *const *arg_names, const char *const *idx_names,
                      char *buf, size_t cap)
{
    if (!plan) return 0;
    std::string text;
    if (guarded([&] { text = print_expression(*plan, which, arg_names, idx_names); }) != TAD_OK || text.empty()) return 0;
    if (buf && cap) {
        size_t n = std::min(cap - 1, text.size());
        std::memcpy(buf, text.data(), n);
        buf[n] = 0;
    }
    return text.size() + 1;
}

tad_status tad_extended_euclid(int64_t a, int64_t b, int64_t *g, int64_t *x, int64_t *y)
{
    return guarded([&] {
        if (!g || !x || !y) throw InvalidArg("NULL argument");
        if (a == 0 && b == 0) throw InvalidArg("gcd(0, 0)");
        extended_euclid(a, b, *g, *x, *y);
    });
}

tad_status tad_smith_normal_form(const int64_t *A, int32_t n_rows, int32_t n_cols,
                                 int64_t *S, int64_t *U, int64_t *V, int32_t *rank)
{
    return guarded([&] {
        if (!A || !S || !U || !V || !rank || n_rows < 1 || n_cols < 1) throw InvalidArg("bad argument");
        Mat m(n_rows, n_cols);
        std::copy(A, A + size_t(n_rows) * n_cols, m.v.begin());
        Smith s = smith_normal_form(m);
        std::copy(s.S.v.begin(), s.S.v.end(), S);
        std::copy(s.U.v.begin(), s.U.v.end(), U);
        std::copy(s.V.v.begin(), s.V.v.end(), V);
        *rank = s.rank;
    });
}

tad_status tad_fourier_motzkin(const int64_t *A, int32_t n_rows, int32_t n_cols, int32_t cap_rows,
                               int32_t *n_lower, int32_t *n_upper,
                               int64_t *L_num, int64_t *Lhat_num, int64_t *L_den,
                               int64_t *H_num, int64_t *Hhat_num, int64_t *H_den,
                               int32_t *n_feas, int64_t *F_num)
{
    return guarded([&] {
        if (!A || !n_lower || !n_upper || !L_num || !Lhat_num || !L_den || !H_num || !Hhat_num || !H_den || !n_feas || !F_num ||
            n_rows < 1 || n_cols < 1 || cap_rows < 1)
            throw InvalidArg("bad argument");
        Mat m(n_rows, n_cols);
        std::copy(A, A + size_t(n_rows) * n_cols, m.v.begin());
        std::vector<int> order;
        for (int k = 0; k < n_cols; ++k) order.push_back(k);   // x_1 first, as in the paper
        FmResult r = fourier_motzkin(m, order, cap_rows);
        for (int k = 0; k < n_cols; ++k) {
            n_lower[k] = (int)r.lower[k].size(); n_upper[k] = (int)r.upper[k].size();
            for (int side = 0; side < 2; ++side) {
                const auto &src = side ? r.upper[k] : r.lower[k];
                int64_t *num = side ? H_num : L_num, *hat = side ? Hhat_num : Lhat_num, *den = side ? H_den : L_den;
                for (int i = 0; i < (int)src.size(); ++i) {
                    size_t row = size_t(k) * cap_rows + i;
                    den[row] = src[i].den;
                    for (int j = 0; j < n_rows; ++j) num[row * n_rows + j] = src[i].bcoef[j];
                    for (int j = 0; j < n_cols; ++j) hat[row * n_cols + j] = src[i].zcoef[j];
                }
            }
        }
        if ((int)r.feas.size() > cap_rows) throw Unsupported("too many feasibility rows");
        *n_feas = (int)r.feas.size();
        for (int i = 0; i < (int)r.feas.size(); ++i)
            for (int j = 0; j < n_rows; ++j) F_num[size_t(i) * n_rows + j] = r.feas[i][j];
    });
}

}  // extern "C"

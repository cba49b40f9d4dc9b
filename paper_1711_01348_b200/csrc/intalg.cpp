// Exact integer algebra (host only).  See intalg.h.
#include "intalg.h"

#include <algorithm>
#include <utility>

namespace tad {

int64_t gcd64(int64_t a, int64_t b)
{
    a = abs_ck(a); b = abs_ck(b);
    while (b) { int64_t t = a % b; a = b; b = t; }
    return a;
}

Mat matmul(const Mat &a, const Mat &b)
{
    Mat c(a.rows, b.cols);
    for (int i = 0; i < a.rows; ++i)
        for (int j = 0; j < b.cols; ++j) {
            int64_t s = 0;
            for (int k = 0; k < a.cols; ++k) s = add_ck(s, mul_ck(a(i, k), b(k, j)));
            c(i, j) = s;
        }
    return c;
}

// Extended Euclidean algorithm (Algorithm "Extended Euclidean algorithm", Sec. 4.1): keeps
// the remainder sequence r and the two cofactor sequences s, t with r_i = |a| s_i + |b| t_i.
// The paper states it for positive inputs; the Smith algorithm calls it on signed entries,
// so it runs on absolute values and the signs move into the factors.
void extended_euclid(int64_t a, int64_t b, int64_t &g, int64_t &x, int64_t &y)
{
    int64_t r0 = abs_ck(a), r1 = abs_ck(b);
    int64_t s0 = 1, s1 = 0, t0 = 0, t1 = 1;
    while (r1 != 0) {
        int64_t q = r0 / r1;                       // operands non-negative: truncation = floor
        int64_t r2 = sub_ck(r0, mul_ck(q, r1));
        int64_t s2 = sub_ck(s0, mul_ck(q, s1));
        int64_t t2 = sub_ck(t0, mul_ck(q, t1));
        r0 = r1; r1 = r2; s0 = s1; s1 = s2; t0 = t1; t1 = t2;
    }
    g = r0;
    x = a < 0 ? neg_ck(s0) : s0;
    y = b < 0 ? neg_ck(t0) : t0;
}

namespace {

void swap_rows(Mat &m, int a, int b) { if (a != b) for (int c = 0; c < m.cols; ++c) std::swap(m(a, c), m(b, c)); }
void swap_cols(Mat &m, int a, int b) { if (a != b) for (int r = 0; r < m.rows; ++r) std::swap(m(r, a), m(r, b)); }

// simultaneously row_a <- s*row_a + t*row_b ; row_b <- u*row_a + v*row_b
void combine_rows(Mat &m, int a, int b, int64_t s, int64_t t, int64_t u, int64_t v)
{
    for (int c = 0; c < m.cols; ++c) {
        int64_t pa = m(a, c), pb = m(b, c);
        m(a, c) = add_ck(mul_ck(s, pa), mul_ck(t, pb));
        m(b, c) = add_ck(mul_ck(u, pa), mul_ck(v, pb));
    }
}
void combine_cols(Mat &m, int a, int b, int64_t s, int64_t t, int64_t u, int64_t v)
{
    for (int r = 0; r < m.rows; ++r) {
        int64_t pa = m(r, a), pb = m(r, b);
        m(r, a) = add_ck(mul_ck(s, pa), mul_ck(t, pb));
        m(r, b) = add_ck(mul_ck(u, pa), mul_ck(v, pb));
    }
}

// Diagonalise the trailing block of S starting at the active index `a`; returns the rank.
int diagonalise(Mat &S, Mat &U, Mat &V, int a)
{
    const int N = S.rows, M = S.cols;
    for (;;) {
        // pivot: non-zero entry of smallest absolute value in the trailing block (ties: row-major)
        int pi = -1, pj = -1;
        for (int i = a; i < N; ++i)
            for (int j = a; j < M; ++j)
                if (S(i, j) != 0 && (pi < 0 || abs_ck(S(i, j)) < abs_ck(S(pi, pj)))) { pi = i; pj = j; }
        if (pi < 0) break;
        swap_cols(S, a, pj); swap_cols(V, a, pj);
        swap_rows(S, a, pi); swap_rows(U, a, pi);
        bool changing = true;
        while (changing) {
            changing = false;
            // rows below the pivot: first make the pivot divide them (Bezout), then subtract multiples
            for (int i = a + 1; i < N; ++i)
                if (S(i, a) % S(a, a) != 0) {
                    int64_t g, sg, tg;
                    extended_euclid(S(a, a), S(i, a), g, sg, tg);
                    int64_t gam = S(i, a) / g, alp = S(a, a) / g;
                    combine_rows(S, a, i, sg, tg, neg_ck(gam), alp);
                    combine_rows(U, a, i, sg, tg, neg_ck(gam), alp);
                    changing = true;
                }
            for (int i = a + 1; i < N; ++i)
                if (S(i, a) != 0) {
                    int64_t f = S(i, a) / S(a, a);
                    combine_rows(S, a, i, 1, 0, neg_ck(f), 1);
                    combine_rows(U, a, i, 1, 0, neg_ck(f), 1);
                    changing = true;
                }
            // columns right of the pivot, likewise
            for (int j = a + 1; j < M; ++j)
                if (S(a, j) % S(a, a) != 0) {
                    int64_t g, sg, tg;
                    extended_euclid(S(a, a), S(a, j), g, sg, tg);
                    int64_t gam = S(a, j) / g, alp = S(a, a) / g;
                    combine_cols(S, a, j, sg, tg, neg_ck(gam), alp);
                    combine_cols(V, a, j, sg, tg, neg_ck(gam), alp);
                    changing = true;
                }
            for (int j = a + 1; j < M; ++j)
                if (S(a, j) != 0) {
                    int64_t f = S(a, j) / S(a, a);
                    combine_cols(S, a, j, 1, 0, neg_ck(f), 1);
                    combine_cols(V, a, j, 1, 0, neg_ck(f), 1);
                    changing = true;
                }
        }
        ++a;
    }
    return a;
}

}  // namespace

// Smith normal form by elementary row and column operations (Algorithm "Smith normal form of
// an integer matrix", Sec. 4.1).  Readings of the points the paper leaves open: the pivot is
// the entry of smallest absolute value; after the divisibility fix-up (adding column a+1 to
// column a) the diagonalisation restarts at index a and the final pass is repeated from the
// first diagonal entry until it changes nothing.  A zero matrix is accepted (rank 0).
Smith smith_normal_form(const Mat &A)
{
    Smith r;
    r.S = A;
    r.U = Mat::identity(A.rows);
    r.V = Mat::identity(A.cols);
    int R = diagonalise(r.S, r.U, r.V, 0);
    for (bool again = true; again;) {
        again = false;
        for (int a = 0; a < R; ++a) {
            if (r.S(a, a) < 0) {
                for (int i = 0; i < r.S.rows; ++i) r.S(i, a) = neg_ck(r.S(i, a));
                for (int i = 0; i < r.V.rows; ++i) r.V(i, a) = neg_ck(r.V(i, a));
            }
            if (a + 1 < R && r.S(a + 1, a + 1) % r.S(a, a) != 0) {
                combine_cols(r.S, a, a + 1, 1, 1, 0, 1);
                combine_cols(r.V, a, a + 1, 1, 1, 0, 1);
                R = diagonalise(r.S, r.U, r.V, a);
                again = true;
                break;
            }
        }
    }
    r.rank = R;
    return r;
}

Mat unimodular_inverse(const Mat &Min)
{
    const int n = Min.rows;
    if (Min.cols != n) throw Unsupported("unimodular_inverse: not square");
    Mat M = Min, I = Mat::identity(n);
    for (int c = 0; c < n; ++c) {
        // gcd-reduce column c over rows >= c into row c
        for (int i = c + 1; i < n; ++i) {
            if (M(i, c) == 0) continue;
            if (M(c, c) == 0) { swap_rows(M, c, i); swap_rows(I, c, i); continue; }
            int64_t g, s, t;
            extended_euclid(M(c, c), M(i, c), g, s, t);
            int64_t gam = M(i, c) / g, alp = M(c, c) / g;
            combine_rows(M, c, i, s, t, neg_ck(gam), alp);
            combine_rows(I, c, i, s, t, neg_ck(gam), alp);
        }
        if (M(c, c) != 1 && M(c, c) != -1) throw Unsupported("unimodular_inverse: determinant is not +-1");
        if (M(c, c) == -1)
            for (int j = 0; j < n; ++j) { M(c, j) = neg_ck(M(c, j)); I(c, j) = neg_ck(I(c, j)); }
        for (int i = 0; i < c; ++i)
            if (M(i, c) != 0) {
                int64_t f = M(i, c);
                combine_rows(M, c, i, 1, 0, neg_ck(f), 1);
                combine_rows(I, c, i, 1, 0, neg_ck(f), 1);
            }
    }
    return I;
}

namespace {

struct WorkRow {
    FmRow r;
    uint64_t hist;   // which original rows were combined into this one
};

void normalise(WorkRow &w)
{
    int64_t g = 0;
    for (int64_t v : w.r.a) g = gcd64(g, v);
    for (int64_t v : w.r.b) g = gcd64(g, v);
    if (g > 1) {
        for (int64_t &v : w.r.a) v /= g;
        for (int64_t &v : w.r.b) v /= g;
    }
}

bool same(const WorkRow &x, const WorkRow &y) { return x.r.a == y.r.a && x.r.b == y.r.b; }

}  // namespace

// Fourier-Motzkin elimination for A z >= beta with symbolic beta (Algorithm "Fourier-Motzkin
// elimination", Sec. 4.2).  The paper divides each row by |A_ik| so that the coefficient of
// the eliminated variable is +-1; here rows stay integer and the positive divisor is kept as
// the bound's denominator, which is the same system scaled by positive factors.  Matrix B of
// the algorithm (which original right-hand sides a row combines) is FmRow::b.  Rows are
// reduced by their gcd and duplicates dropped; a row that combines more than (number of
// eliminations + 1) original rows is redundant (Chernikov's rule) and dropped.
FmResult fourier_motzkin(const Mat &A, const std::vector<int> &order, int max_rows)
{
    const int N = A.rows, M = A.cols;
    if (N > 64) throw Unsupported("fourier_motzkin: more than 64 inequalities");
    FmResult out;
    out.lower.resize(M);
    out.upper.resize(M);
    std::vector<WorkRow> rows(N);
    for (int i = 0; i < N; ++i) {
        rows[i].r.a.resize(M);
        rows[i].r.b.assign(N, 0);
        for (int j = 0; j < M; ++j) rows[i].r.a[j] = A(i, j);
        rows[i].r.b[i] = 1;
        rows[i].hist = uint64_t(1) << i;
    }
    int eliminations = 0;
    for (int k : order) {
        std::vector<int> zero, pos, neg;
        for (int i = 0; i < (int)rows.size(); ++i)
            (rows[i].r.a[k] == 0 ? zero : rows[i].r.a[k] > 0 ? pos : neg).push_back(i);
        for (int i : pos) {          // z_k >= (b.beta - sum_{j != k} a_j z_j) / a_k
            FmBound bd;
            bd.den = rows[i].r.a[k];
            bd.bcoef = rows[i].r.b;
            bd.zcoef.assign(M, 0);
            for (int j = 0; j < M; ++j) if (j != k) bd.zcoef[j] = neg_ck(rows[i].r.a[j]);
            out.lower[k].push_back(bd);
        }
        for (int i : neg) {          // z_k <= (-b.beta + sum_{j != k} a_j z_j) / (-a_k)
            FmBound bd;
            bd.den = neg_ck(rows[i].r.a[k]);
            bd.bcoef.resize(N);
            for (int j = 0; j < N; ++j) bd.bcoef[j] = neg_ck(rows[i].r.b[j]);
            bd.zcoef.assign(M, 0);
            for (int j = 0; j < M; ++j) if (j != k) bd.zcoef[j] = rows[i].r.a[j];
            out.upper[k].push_back(bd);
        }
        std::vector<WorkRow> next;
        for (int i : zero) next.push_back(rows[i]);
        if (!pos.empty() && !neg.empty()) {
            ++eliminations;
            for (int p : pos)
                for (int n : neg) {
                    WorkRow w;
                    int64_t fp = neg_ck(rows[n].r.a[k]), fn = rows[p].r.a[k];   // both > 0
                    w.r.a.resize(M);
                    w.r.b.resize(N);
                    for (int j = 0; j < M; ++j)
                        w.r.a[j] = add_ck(mul_ck(fp, rows[p].r.a[j]), mul_ck(fn, rows[n].r.a[j]));
                    for (int j = 0; j < N; ++j)
                        w.r.b[j] = add_ck(mul_ck(fp, rows[p].r.b[j]), mul_ck(fn, rows[n].r.b[j]));
                    w.hist = rows[p].hist | rows[n].hist;
                    if (__builtin_popcountll(w.hist) > eliminations + 1) continue;
                    normalise(w);
                    bool dup = false;
                    for (const WorkRow &o : next) if (same(o, w)) { dup = true; break; }
                    if (!dup) next.push_back(std::move(w));
                    if ((int)next.size() > max_rows * 8) throw Unsupported("fourier_motzkin: too many rows");
                }
        }
        // one-sided or absent variable: rows that contain it are dropped (nothing to combine)
        rows.swap(next);
    }
    for (const WorkRow &w : rows) out.feas.push_back(w.r.b);   // 0 >= b.beta  <=>  F beta <= 0
    for (int k = 0; k < M; ++k)
        if ((int)out.lower[k].size() > max_rows || (int)out.upper[k].size() > max_rows)
            throw Unsupported("fourier_motzkin: too many bound rows");
    return out;
}

}  // namespace tad

// Exact integer algebra on small int64 matrices (host only): extended Euclid, Smith
// normal form (Sec. 4.1 of the paper) and Fourier-Motzkin elimination (Sec. 4.2).
// Every multiplication and addition is overflow-checked; an overflow throws tad::Overflow.
#pragma once
#include <cstdint>
#include <stdexcept>
#include <string>
#include <vector>

namespace tad {

struct Overflow : std::runtime_error {
    Overflow() : std::runtime_error("integer overflow in exact arithmetic") {}
};
struct Unsupported : std::runtime_error {
    explicit Unsupported(const std::string &m) : std::runtime_error(m) {}
};

inline int64_t mul_ck(int64_t a, int64_t b) { int64_t r; if (__builtin_mul_overflow(a, b, &r)) throw Overflow(); return r; }
inline int64_t add_ck(int64_t a, int64_t b) { int64_t r; if (__builtin_add_overflow(a, b, &r)) throw Overflow(); return r; }
inline int64_t sub_ck(int64_t a, int64_t b) { int64_t r; if (__builtin_sub_overflow(a, b, &r)) throw Overflow(); return r; }
inline int64_t neg_ck(int64_t a) { return sub_ck(0, a); }
inline int64_t abs_ck(int64_t a) { return a < 0 ? neg_ck(a) : a; }

// floor and ceiling of a / b for b > 0 (C division truncates toward zero)
inline int64_t floor_div(int64_t a, int64_t b) { int64_t q = a / b; return (a % b != 0 && a < 0) ? q - 1 : q; }
inline int64_t ceil_div(int64_t a, int64_t b) { int64_t q = a / b; return (a % b != 0 && a > 0) ? q + 1 : q; }

int64_t gcd64(int64_t a, int64_t b);   // non-negative, gcd(0,0) = 0

// Row-major dense integer matrix.
struct Mat {
    int rows = 0, cols = 0;
    std::vector<int64_t> v;
    Mat() = default;
    Mat(int r, int c) : rows(r), cols(c), v(size_t(r) * c, 0) {}
    int64_t &operator()(int r, int c) { return v[size_t(r) * cols + c]; }
    int64_t operator()(int r, int c) const { return v[size_t(r) * cols + c]; }
    static Mat identity(int n) { Mat m(n, n); for (int i = 0; i < n; ++i) m(i, i) = 1; return m; }
};
Mat matmul(const Mat &a, const Mat &b);

// Bezout factors: g = gcd(a, b) = a x + b y for any signs of a, b (not both zero);
// the extended Euclidean algorithm runs on |a|, |b| and the signs are folded into x, y.
void extended_euclid(int64_t a, int64_t b, int64_t &g, int64_t &x, int64_t &y);

// Smith normal form S = U A V with positive invariant factors, each dividing the next.
struct Smith {
    Mat S, U, V;
    int rank = 0;
};
Smith smith_normal_form(const Mat &A);

// Exact inverse of a unimodular matrix (|det| = 1).
Mat unimodular_inverse(const Mat &M);

// One inequality of a Fourier-Motzkin system:  sum_j a[j] z_j  >=  sum_i b[i] beta_i
// where beta is the symbolic right-hand side vector (one entry per original row).
struct FmRow {
    std::vector<int64_t> a;   // over the M variables
    std::vector<int64_t> b;   // over the N original right-hand sides
};
// Bounds of one variable after elimination of all variables that come earlier in `order`:
// value = (bcoef . beta + sum_j zcoef[j] z_j) / den, den > 0; a lower row means z_k >= value,
// an upper row z_k <= value.  zcoef is zero at k and at every variable eliminated before k.
struct FmBound {
    int64_t den;
    std::vector<int64_t> bcoef;   // N
    std::vector<int64_t> zcoef;   // M
};
struct FmResult {
    std::vector<std::vector<FmBound>> lower, upper;   // indexed by variable
    std::vector<std::vector<int64_t>> feas;           // rows F: system feasible iff F beta <= 0
};
// Eliminates variables in the given order (order[0] first = innermost loop).
FmResult fourier_motzkin(const Mat &A, const std::vector<int> &order, int max_rows);

}  // namespace tad

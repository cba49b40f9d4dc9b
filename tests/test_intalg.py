"""Host integer algebra of the library (extended Euclid, Smith normal form, Fourier-Motzkin)
against what the mathematics fixes: invariants, gcds of minors, brute-force point sets and the
paper's lattice figures.  Host only: no GPU call."""
import itertools
import math
import os
import random

import numpy as np
import pytest

from paper_1711_01348_b200 import extended_euclid, fourier_motzkin, smith_normal_form, TadError


def test_extended_euclid_bezout():
    rnd = random.Random(7)
    for _ in range(500):
        a, b = rnd.randint(-10**6, 10**6), rnd.randint(-10**6, 10**6)
        if a == 0 and b == 0:
            continue
        g, x, y = extended_euclid(a, b)
        assert g == math.gcd(a, b)
        assert a * x + b * y == g
    assert extended_euclid(240, 46) [0] == 2
    with pytest.raises(TadError):
        extended_euclid(0, 0)


def _det(M):
    return round(np.linalg.det(np.array(M, dtype=np.float64)))


def _minor_gcd(A, k):
    A = np.array(A, dtype=object)
    g = 0
    for rows in itertools.combinations(range(A.shape[0]), k):
        for cols in itertools.combinations(range(A.shape[1]), k):
            sub = np.array(A[np.ix_(rows, cols)], dtype=np.float64)
            g = math.gcd(g, int(round(np.linalg.det(sub))))
    return g


def _check_snf(A):
    S, U, V, R = smith_normal_form(A)
    A_, S_, U_, V_ = (np.array(m, dtype=object) for m in (A, S, U, V))
    assert (U_.dot(A_).dot(V_) == S_).all()
    assert abs(_det(U)) == 1 and abs(_det(V)) == 1
    n, m = A_.shape
    for i in range(n):
        for j in range(m):
            if i != j:
                assert S_[i, j] == 0
    diag = [S_[i, i] for i in range(min(n, m))]
    assert all(d > 0 for d in diag[:R]) and all(d == 0 for d in diag[R:])
    for i in range(R - 1):
        assert diag[i + 1] % diag[i] == 0
    assert R == np.linalg.matrix_rank(np.array(A, dtype=np.float64))
    # uniqueness of S: the product of the first k invariant factors is the gcd of the k x k minors
    prod = 1
    for k in range(1, R + 1):
        prod *= diag[k - 1]
        assert prod == _minor_gcd(A, k)
    # kernel and pseudo-inverse properties: A K = 0 and A (V S^+ U) A = A
    K = V_[:, R:]
    assert (A_.dot(K) == 0).all()
    from fractions import Fraction
    Splus = np.zeros((m, n), dtype=object)
    for i in range(R):
        Splus[i, i] = Fraction(1, int(diag[i]))
    I = V_.dot(Splus).dot(U_)
    assert (A_.dot(I).dot(A_) == A_).all()
    return S, U, V, R


def test_smith_normal_form_random():
    rnd = random.Random(11)
    for _ in range(300):
        n, m = rnd.randint(1, 4), rnd.randint(1, 5)
        A = [[rnd.randint(-6, 6) for _ in range(m)] for _ in range(n)]
        if rnd.random() < 0.3 and n > 1:      # force rank deficiency
            A[-1] = [2 * v for v in A[0]]
        _check_snf(A)


def test_smith_normal_form_known():
    # classic example with invariant factors 2, 2, 156
    S, _, _, R = _check_snf([[2, 4, 4], [-6, 6, 12], [10, 4, 16]])
    assert [S[i][i] for i in range(3)] == [2, 2, 156] and R == 3
    # needs the divisibility fix-up: diag(2, 3) -> diag(1, 6)
    S, _, _, R = _check_snf([[2, 0], [0, 3]])
    assert [S[0][0], S[1][1]] == [1, 6]
    S, _, _, R = _check_snf([[4, 0, 0], [0, 6, 0], [0, 0, 9]])
    assert [S[i][i] for i in range(3)] == [1, 6, 36]
    S, _, _, R = _check_snf([[0, 0], [0, 0]])
    assert R == 0
    # the index maps of the workloads
    S, _, _, R = _check_snf([[2, 1, 0], [0, 1, -1]])
    assert [S[0][0], S[1][1]] == [1, 1]
    S, _, _, R = _check_snf([[0, 0, 3]])
    assert S[0][0] == 3 and R == 1
    S, _, _, R = _check_snf([[2, 4]])
    assert S[0][0] == 2


def _points(A, b, lo=-8, hi=8):
    A = np.array(A); b = np.array(b)
    m = A.shape[1]
    return {z for z in itertools.product(range(lo, hi + 1), repeat=m) if (A.dot(np.array(z)) >= b).all()}


def _walk(bounds, b, m):
    """Enumerate integer points from the bound rows, z_M outermost .. z_1 innermost."""
    out = set()

    def rec(k, z):
        if k < 0:
            out.add(tuple(z))
            return
        lower, upper = bounds[k]
        lo, hi = -10**9, 10**9
        for den, bc, zc in lower:
            num = sum(c * v for c, v in zip(bc, b)) + sum(c * v for c, v in zip(zc, z))
            lo = max(lo, -((-num) // den))
        for den, bc, zc in upper:
            num = sum(c * v for c, v in zip(bc, b)) + sum(c * v for c, v in zip(zc, z))
            hi = min(hi, num // den)
        for v in range(lo, hi + 1):
            z[k] = v
            rec(k - 1, z)
        z[k] = 0

    rec(m - 1, [0] * m)
    return out


def test_fourier_motzkin_matches_brute_force():
    rnd = random.Random(5)
    for trial in range(150):
        m = rnd.randint(1, 3)
        n_extra = rnd.randint(0, 3)
        # a bounded system: a box plus random extra rows
        A, b = [], []
        for j in range(m):
            row = [0] * m; row[j] = 1
            A.append(row); b.append(rnd.randint(-4, 0))
            row = [0] * m; row[j] = -1
            A.append(row); b.append(-rnd.randint(0, 4))
        for _ in range(n_extra):
            A.append([rnd.randint(-3, 3) for _ in range(m)]); b.append(rnd.randint(-6, 2))
        bounds, feas = fourier_motzkin(A)
        want = _points(A, b, -5, 5)
        feasible_real = all(sum(c * v for c, v in zip(f, b)) <= 0 for f in feas)
        if not feasible_real:
            assert not want
        got = _walk(bounds, b, m) if feasible_real else set()
        assert got == want, (A, b)
        # bound rows of variable k only read later variables
        for k, (lower, upper) in enumerate(bounds):
            for den, bc, zc in lower + upper:
                assert den > 0 and all(c == 0 for c in zc[:k + 1])


def _golden(path):
    rows = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        tok = line.split()
        rows.setdefault(tok[0], []).append(tok[1:])
    return rows


def test_figure1_one_dimensional_kernel(golden_dir):
    g = _golden(os.path.join(golden_dir, "fig1_lattice.txt"))
    A = [[int(v) for v in g["A"][0]]]
    lo = [int(v) for v in g["box_lo"][0]]; hi = [int(v) for v in g["box_hi"][0]]
    beta = int(g["beta"][0][0])
    S, U, V, R = smith_normal_form(A)
    assert R == 1 and S[0][0] == 1
    K = [V[0][1], V[1][1]]
    assert A[0][0] * K[0] + A[0][1] * K[1] == 0 and sorted(map(abs, K)) == [1, 2]   # +-(2, 1)
    # alpha = x' V[:,0] + z K with x' = U beta; constraints lo <= alpha <= hi in z
    x = U[0][0] * beta
    a0 = [V[0][0] * x, V[1][0] * x]
    rows = [[K[0]], [K[1]], [-K[0]], [-K[1]]]
    b = [lo[0] - a0[0], lo[1] - a0[1], a0[0] - hi[0], a0[1] - hi[1]]
    bounds, feas = fourier_motzkin(rows)
    zs = _walk(bounds, b, 1)
    pts = sorted((a0[0] + K[0] * z[0], a0[1] + K[1] * z[0]) for z in zs)
    want = [int(v) for v in g["points"][0]]
    assert pts == [(want[0], want[1]), (want[2], want[3]), (want[4], want[5])]
    assert len(zs) == int(g["z_range"][0][1]) - int(g["z_range"][0][0]) + 1


def test_figure2_two_dimensional_kernel(golden_dir):
    g = _golden(os.path.join(golden_dir, "fig2_lattice.txt"))
    A = [[int(v) for v in r[:2]] for r in g["ineq"]]
    b = [int(r[2]) for r in g["ineq"]]
    bounds, feas = fourier_motzkin(A)        # z1 innermost, z2 outermost
    pts = _walk(bounds, b, 2)
    assert len(pts) == int(g["n_points"][0][0])
    z2lo, z2hi = (int(v) for v in g["z2_range"][0])
    assert {p[1] for p in pts} == set(range(z2lo, z2hi + 1))
    for z2 in range(z2lo, z2hi + 1):
        z1 = sorted(p[0] for p in pts if p[1] == z2)
        assert z1 == list(range(max(-1, -z2), min(1, 4 - z2) + 1))

"""Pins for the CPU oracle: closed forms from the paper, library routines, finite
differences and brute force.  None of these re-use the oracle's own code; each is
an independent statement of what the result must be."""
import os

import numpy as np
import pytest
import torch

from oracle.oracle import Oracle, max_threads
from workloads import configs as W

RNG = np.random.default_rng(1234)


def rnd(*shape):
    return RNG.uniform(-0.9, 0.9, size=shape)


# --------------------------------------------------------------------------- #
# Sec. 1 examples
# --------------------------------------------------------------------------- #

def test_square_broadcast_sec1():
    # f_ij = x_i^2  =>  dx_i = sum_j df_ij 2 x_i
    ni, nj = 5, 7
    x, df = rnd(ni), rnd(ni, nj)
    o = Oracle(W.ex_square_broadcast(ni, nj))
    f, fabs = o.forward([x])
    np.testing.assert_allclose(f, np.repeat((x ** 2)[:, None], nj, 1), rtol=1e-15)
    np.testing.assert_allclose(fabs, np.abs(f), rtol=1e-15)
    (dx,), (tb,) = o.backward([x], df)
    np.testing.assert_allclose(dx, df.sum(1) * 2 * x, rtol=1e-13)
    np.testing.assert_allclose(tb, np.abs(df * 2 * x[:, None]).sum(1), rtol=1e-13)
    np.testing.assert_array_equal(o.counts(0), np.full(ni, nj))


def test_diag_square_sec1():
    # f_i = x_ii^2  =>  dx_ij = delta_ij df_i 2 x_ii
    n = 6
    x, df = rnd(n, n), rnd(n)
    o = Oracle(W.ex_diag_square(n))
    f, _ = o.forward([x])
    np.testing.assert_allclose(f, np.diag(x) ** 2, rtol=1e-15)
    (dx,), _ = o.backward([x], df)
    np.testing.assert_allclose(dx, np.diag(df * 2 * np.diag(x)), rtol=1e-14)
    np.testing.assert_array_equal(o.counts(0), np.eye(n, dtype=np.int64))


def test_exp_shift_sec1():
    # f_ij = exp x_{i+j}  =>  dx_k = sum_i df_{i,k-i} exp x_k, i restricted so that 0 <= k-i < nj
    ni, nj = 4, 6
    x, df = rnd(ni + nj - 1), rnd(ni, nj)
    o = Oracle(W.ex_exp_shift(ni, nj))
    f, _ = o.forward([x])
    for i in range(ni):
        for j in range(nj):
            assert f[i, j] == pytest.approx(np.exp(x[i + j]), rel=1e-15)
    (dx,), _ = o.backward([x], df)
    want = np.zeros_like(x)
    cnt = np.zeros(len(x), dtype=np.int64)
    for k in range(len(x)):
        for i in range(max(0, k - nj + 1), min(ni - 1, k) + 1):
            want[k] += df[i, k - i] * np.exp(x[k])
            cnt[k] += 1
    np.testing.assert_allclose(dx, want, rtol=1e-13)
    np.testing.assert_array_equal(o.counts(0), cnt)


# --------------------------------------------------------------------------- #
# Sec. 5 examples f^1 ... f^5
# --------------------------------------------------------------------------- #

def test_f1_sin():
    n = 9
    x, dg = rnd(n), rnd(n)
    o = Oracle(W.ex_sin(n))
    np.testing.assert_allclose(o.forward([x])[0], np.sin(x), rtol=1e-15)
    np.testing.assert_allclose(o.backward([x], dg)[0][0], dg * np.cos(x), rtol=1e-14)


def test_f2_xy():
    n = 5
    x, y, dg = rnd(n), rnd(n, n), rnd(n, n)
    o = Oracle(W.ex_xy(n))
    np.testing.assert_allclose(o.forward([x, y])[0], x[:, None] * y, rtol=1e-15)
    (dx, dy), _ = o.backward([x, y], dg)
    np.testing.assert_allclose(dx, (dg * y).sum(1), rtol=1e-13)
    np.testing.assert_allclose(dy, dg * x[:, None], rtol=1e-14)


def test_f3_diag_cube():
    n = 5
    x, dg = rnd(n, n), rnd(n)
    o = Oracle(W.ex_diag_cube(n))
    np.testing.assert_allclose(o.forward([x])[0], np.diag(x) ** 3, rtol=1e-14)
    np.testing.assert_allclose(o.backward([x], dg)[0][0], np.diag(dg * 3 * np.diag(x) ** 2), rtol=1e-14)


def test_f4_matmul_is_gemm():
    ni, nk, nj = 4, 6, 5
    x, y, dg = rnd(ni, nk), rnd(nk, nj), rnd(ni, nj)
    o = Oracle(W.ex_matmul(ni, nk, nj))
    f, fabs = o.forward([x, y])
    np.testing.assert_allclose(f, x @ y, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(fabs, np.abs(x) @ np.abs(y), rtol=1e-13)
    (dx, dy), (tx, ty) = o.backward([x, y], dg)
    np.testing.assert_allclose(dx, dg @ y.T, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(dy, x.T @ dg, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(tx, np.abs(dg) @ np.abs(y).T, rtol=1e-13)
    np.testing.assert_array_equal(o.counts(0), np.full((ni, nk), nj))
    np.testing.assert_array_equal(o.counts(1), np.full((nk, nj), ni))


def test_f5_exp_flat():
    n, m = 4, 3
    x, dg = rnd(n * m), rnd(n, m)
    o = Oracle(W.ex_exp_flat(n, m))
    np.testing.assert_allclose(o.forward([x])[0], np.exp(x).reshape(n, m), rtol=1e-15)
    # dx_{i'} = sum_i dg_{i, i'-Mi} exp x_{i'}: exactly one i has 0 <= i'-Mi < M
    np.testing.assert_allclose(o.backward([x], dg)[0][0], dg.reshape(-1) * np.exp(x), rtol=1e-14)


# --------------------------------------------------------------------------- #
# Sec. 6: the derivative expressions the paper prints, retyped with their ranges
# --------------------------------------------------------------------------- #

def _sec6_inputs():
    a, b, c, d = rnd(3, 5), rnd(4, 5), rnd(3, 3), rnd(8)
    df = rnd(3, 4)
    return a, b, c, d, df


def _sec6_S(a, b, c, d, i, j):
    return sum((a[i, k] + b[j, k]) ** 2 * c[i, i] + d[i + k] ** 3 for k in range(5))


def test_section6_printed_derivatives(golden_dir):
    a, b, c, d, df = _sec6_inputs()
    o = Oracle(W.ex_section6())
    f, _ = o.forward([a, b, c, d])
    for i in range(3):
        for j in range(4):
            assert f[i, j] == pytest.approx(np.exp(-_sec6_S(a, b, c, d, i, j)), rel=1e-14)
    (da, db, dc, dd), _ = o.backward([a, b, c, d], df)

    def g(i, j):   # -(df[i;j] * exp(-sum ...)) as printed
        return -(df[i, j] * np.exp(-_sec6_S(a, b, c, d, i, j)))

    want_da = np.zeros((3, 5)); want_db = np.zeros((4, 5)); want_dc = np.zeros((3, 3)); want_dd = np.zeros(8)
    for i0 in range(3):
        for i1 in range(5):
            want_da[i0, i1] = sum(g(i0, z0) * c[i0, i0] * 2 * (a[i0, i1] + b[z0, i1]) for z0 in range(0, 3 + 1))
    for j0 in range(4):
        for j1 in range(5):
            want_db[j0, j1] = sum(g(z0, j0) * c[z0, z0] * 2 * (a[z0, j1] + b[j0, j1]) for z0 in range(0, 2 + 1))
    for c0 in range(3):
        for c1 in range(3):
            if c0 - c1 == 0:
                want_dc[c0, c1] = sum((a[c1, z1] + b[z0, z1]) ** 2 * g(c1, z0)
                                      for z1 in range(0, 4 + 1) for z0 in range(0, 3 + 1))
    for d0 in range(8):
        for z1 in range(max(0, -2 + d0), min(4, d0) + 1):
            for z0 in range(0, 3 + 1):
                want_dd[d0] += g(d0 - z1, z0) * 3 * d[d0] ** 2
    np.testing.assert_allclose(da, want_da, rtol=1e-12)
    np.testing.assert_allclose(db, want_db, rtol=1e-12)
    np.testing.assert_allclose(dc, want_dc, rtol=1e-12)
    np.testing.assert_allclose(dd, want_dd, rtol=1e-12, atol=1e-300)
    assert dd[7] == 0.0   # d has 8 elements, i+k <= 6: the printed range 5..4 is empty

    # term counts printed implicitly by the ranges (golden file)
    golden = {}
    for line in open(os.path.join(golden_dir, "section6_ranges.txt")):
        if line.startswith("#") or not line.strip():
            continue
        tok = line.split()
        if tok[1] == "counts":
            golden[tok[0]] = [int(t) for t in tok[2:]]
    e = o.expr
    acc_of = {e.arg_names[a_.arg]: q for q, a_ in enumerate(e.accesses)}
    np.testing.assert_array_equal(o.counts(acc_of["d"]), np.array(golden["dd"]))
    np.testing.assert_array_equal(o.counts(acc_of["a"]), np.full((3, 5), 4))
    np.testing.assert_array_equal(o.counts(acc_of["b"]), np.full((4, 5), 3))
    np.testing.assert_array_equal(o.counts(acc_of["c"]), 20 * np.eye(3, dtype=np.int64))


# --------------------------------------------------------------------------- #
# the paper's own experiment (Sec. 6): numeric differentiation on random inputs
# --------------------------------------------------------------------------- #

def _finite_difference_check(e, args, df, eps=1e-6, rtol=2e-6):
    o = Oracle(e)
    dx, _ = o.backward(args, df)
    for p, x in enumerate(args):
        flat = x.reshape(-1)
        for idx in range(flat.size):
            keep = flat[idx]
            flat[idx] = keep + eps
            lp = float((o.forward(args)[0] * df).sum())
            flat[idx] = keep - eps
            lm = float((o.forward(args)[0] * df).sum())
            flat[idx] = keep
            num = (lp - lm) / (2 * eps)
            got = dx[p].reshape(-1)[idx]
            assert got == pytest.approx(num, rel=rtol, abs=2e-8), (e.name, p, idx, got, num)


@pytest.mark.parametrize("make", [
    lambda: W.ex_all_ops(3),
    lambda: W.ex_section6(),
    lambda: W.shifted(3),
    lambda: W.nonunimodular(3),
    lambda: W.conv1d(2, 2, 3, 4, 5),
    lambda: W.ex_strided(4, 2),
    lambda: W.ex_strided2(3, 3),
    lambda: W.ex_lattice2d(3, 3),
])
def test_numeric_differentiation(make):
    e = make()
    args = [rnd(*s) for s in e.arg_shapes]
    df = rnd(*e.out_shape)
    _finite_difference_check(e, args, df)


# --------------------------------------------------------------------------- #
# second opinion: float64 torch autograd over explicit index tensors
# --------------------------------------------------------------------------- #

def _torch_grads(fn, args, df):
    ts = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in args]
    f = fn(*ts)
    (f * torch.tensor(df)).sum().backward()
    return f.detach().numpy(), [t.grad.numpy() if t.grad is not None else np.zeros_like(a)
                                for t, a in zip(ts, args)]


def _compare_with_torch(e, fn, seed=0):
    r = np.random.default_rng(seed)
    args = [r.uniform(-0.8, 0.8, size=s) for s in e.arg_shapes]
    df = r.normal(size=e.out_shape)
    o = Oracle(e)
    f, _ = o.forward(args)
    dx, tb = o.backward(args, df)
    f_t, dx_t = _torch_grads(fn, args, df)
    np.testing.assert_allclose(f, f_t, rtol=1e-12, atol=1e-14)
    for got, want, t in zip(dx, dx_t, tb):
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)
        assert np.all(np.abs(got) <= t * (1 + 1e-12) + 1e-300)


def test_intro_structure_vs_autograd():
    ni, nj, nk = 5, 4, 3
    e = W.intro(ni, nj, nk)

    def fn(a, b, c, d):
        i = torch.arange(ni)
        k = torch.arange(nk)
        s = ((a[:, None, :] + b[None, :, :]) ** 2 * torch.diagonal(c)[:, None, None]
             + (d[i[:, None] + k[None, :]] ** 3)[:, None, :]).sum(-1)
        return torch.exp(-s)
    _compare_with_torch(e, fn)


def test_shifted_structure_vs_autograd():
    n = 6
    e = W.shifted(n)

    def fn(x, w):
        i = torch.arange(n)[:, None]
        j = torch.arange(n)[None, :]
        return torch.exp(x[i + j]) * torch.tanh(x[2 * i + 3 * j]) * torch.diagonal(w)[:, None]
    _compare_with_torch(e, fn)


def test_nonunimodular_structure_vs_autograd():
    n = 4
    e = W.nonunimodular(n)

    def fn(x, y):
        i = torch.arange(n)[:, None, None]
        j = torch.arange(n)[None, :, None]
        k = torch.arange(n)[None, None, :]
        return torch.sin(x[2 * i + j, j - k + n - 1]) * y[3 * k] ** 2
    _compare_with_torch(e, fn)


def test_conv_structure_is_library_conv1d():
    nb, nc, no, nt, nu = 2, 3, 4, 6, 5
    e = W.conv1d(nb, nc, no, nt, nu)

    def fn(x, w):
        return torch.nn.functional.conv1d(x, w, stride=2)
    _compare_with_torch(e, fn)


# --------------------------------------------------------------------------- #
# invariants that hold at any size
# --------------------------------------------------------------------------- #

@pytest.mark.parametrize("key", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_counts_sum_to_box_and_subboxes_add_up(key):
    e = {"cfg1": lambda: W.intro(6, 5, 3), "cfg2": lambda: W.intro(7, 4, 2),
         "cfg3": lambda: W.shifted(7), "cfg4": lambda: W.nonunimodular(4),
         "cfg5": lambda: W.conv1d(2, 3, 2, 5, 5)}[key]()
    o = Oracle(e)
    nf = int(np.prod(e.out_shape))
    sum_ext = {n.sum_idx: n.sum_hi - n.sum_lo + 1 for n in e.nodes if n.op == "sum"}
    for q, a in enumerate(e.accesses):
        # every alpha_hat of the (enclosing) box reads exactly one element
        size = nf
        for idx, ext in sum_ext.items():
            size *= ext   # in these workloads every load sits inside every sum
        assert int(o.counts(q).sum()) == size
    args, df = W.make_inputs(e, ("uniform", -0.5, 0.5), seed=3)
    full_f, _ = o.forward(args)
    full_dx, full_t = o.backward(args, df)
    cut = e.out_shape[0] // 2
    lo0, hi0 = [0] * len(e.out_shape), [cut] + e.out_shape[1:]
    lo1, hi1 = [cut] + [0] * (len(e.out_shape) - 1), list(e.out_shape)
    f0, _ = o.forward(args, lo0, hi0)
    f1, _ = o.forward(args, lo1, hi1)
    np.testing.assert_array_equal(f0 + f1, full_f)
    d0, t0 = o.backward(args, df, lo0, hi0)
    d1, t1 = o.backward(args, df, lo1, hi1)
    for p in range(len(args)):
        np.testing.assert_allclose(d0[p] + d1[p], full_dx[p], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(t0[p] + t1[p], full_t[p], rtol=1e-12, atol=1e-14)


def test_closed_form_counts_shifted():
    n = 9
    e = W.shifted(n)
    o = Oracle(e)
    L = e.arg_shapes[0][0]
    beta = np.arange(L)
    c0 = np.clip(np.minimum(beta, n - 1) - np.maximum(0, beta - n + 1) + 1, 0, None)
    np.testing.assert_array_equal(o.counts(0), c0)
    # 2i + 3j = beta: brute force with a different loop structure (over j, solve for i)
    c1 = np.zeros(L, dtype=np.int64)
    for bt in range(L):
        for j in range(n):
            r = bt - 3 * j
            if r >= 0 and r % 2 == 0 and r // 2 < n:
                c1[bt] += 1
    np.testing.assert_array_equal(o.counts(1), c1)
    np.testing.assert_array_equal(o.counts(2), n * np.eye(n, dtype=np.int64))


def test_parallel_run_matches_single_thread():
    e = W.intro(23, 17, 4)
    args, df = W.make_inputs(e, ("uniform", -0.5, 0.5), seed=5)
    o = Oracle(e)
    f1, _ = o.forward(args, nthreads=1)
    fn, _ = o.forward(args, nthreads=max(2, max_threads()))
    np.testing.assert_array_equal(f1, fn)
    d1, t1 = o.backward(args, df, nthreads=1)
    dn, tn = o.backward(args, df, nthreads=max(2, max_threads()))
    for a, b in zip(d1 + t1, dn + tn):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-15)


def test_out_of_range_access_is_reported():
    e = W.ex_exp_shift(4, 4)
    e.arg_shapes[0] = [5]          # i + j reaches 6
    o = Oracle(e)
    with pytest.raises(RuntimeError):
        o.forward([np.zeros(5)])

"""Seeded synthetic workloads: expression descriptions plus input tensors.

The paper measures on no dataset; these five workloads stand in for one.  Each
builder returns an ``Expr`` (data only) and ``make_inputs`` draws the argument
tensors and the upstream gradient ``df`` as fp32 from a seeded CPU generator, in
declaration order of the arguments and ``df`` last.  Nothing here evaluates an
expression.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import torch

from .expr import Builder, Expr, unit


# --------------------------------------------------------------------------- #
# expression builders (sizes are parameters so that tests can use reduced cases)
# --------------------------------------------------------------------------- #

def intro(ni: int, nj: int, nk: int, c_cols: int | None = None, d_len: int | None = None,
          name: str = "intro") -> Expr:
    """f_ij = exp(-sum_k ((a_ik + b_jk)^2 c_ii + d_{i+k}^3))  (Sec. 1, Sec. 6)."""
    c_cols = ni if c_cols is None else c_cols
    d_len = ni + nk - 1 if d_len is None else d_len
    b = Builder(name, [ni, nj], 1, ["a", "b", "c", "d"],
                [[ni, nk], [nj, nk], [ni, c_cols], [d_len]])
    n = 3  # alpha_hat = (i, j, k)
    a_ik = b.load("a", [unit(n, (0, 1)), unit(n, (2, 1))])
    b_jk = b.load("b", [unit(n, (1, 1)), unit(n, (2, 1))])
    c_ii = b.load("c", [unit(n, (0, 1)), unit(n, (0, 1))])
    d_ik = b.load("d", [unit(n, (0, 1), (2, 1))])
    s = b.bin("add", a_ik, b_jk)
    s2 = b.powi(s, 2)
    t1 = b.bin("mul", s2, c_ii)
    d3 = b.powi(d_ik, 3)
    body = b.bin("add", t1, d3)
    sm = b.sum(2, 0, nk - 1, body)
    b.un("exp", b.un("neg", sm))
    return b.done()


def shifted(n: int, x_len: int | None = None, name: str = "shifted") -> Expr:
    """f_ij = exp(x_{i+j}) * tanh(x_{2i+3j}) * W_ii,  i, j in [0, n)."""
    x_len = 5 * (n - 1) + 3 if x_len is None else x_len
    b = Builder(name, [n, n], 0, ["x", "W"], [[x_len], [n, n]])
    x1 = b.load("x", [unit(2, (0, 1), (1, 1))])
    x2 = b.load("x", [unit(2, (0, 2), (1, 3))])
    w = b.load("W", [unit(2, (0, 1)), unit(2, (0, 1))])
    b.bin("mul", b.bin("mul", b.un("exp", x1), b.un("tanh", x2)), w)
    return b.done()


def nonunimodular(n: int, name: str = "nonunimodular") -> Expr:
    """f_ijk = sin(x_{2i+j, j-k+n-1}) * y_{3k}^2,  i, j, k in [0, n)."""
    b = Builder(name, [n, n, n], 0, ["x", "y"], [[3 * n - 1, 2 * n - 1], [3 * n - 2]])
    x = b.load("x", [unit(3, (0, 2), (1, 1)), unit(3, (1, 1), (2, -1))], [0, n - 1])
    y = b.load("y", [unit(3, (2, 3))])
    b.bin("mul", b.un("sin", x), b.powi(y, 2))
    return b.done()


def conv1d(nb: int, nc: int, no: int, nt: int, nu: int, name: str = "conv1d") -> Expr:
    """f_{b,o,t} = sum_c sum_u w_{o,c,u} x_{b,c,2t+u}  (stride-2 convolution)."""
    x_len = 2 * (nt - 1) + nu + 0
    # the full-size workload pads x by a few unread columns, like the paper's d in Sec. 6
    b = Builder(name, [nb, no, nt], 2, ["x", "w"], [[nb, nc, x_len + 0], [no, nc, nu]])
    n = 5  # alpha_hat = (b, o, t, c, u)
    w = b.load("w", [unit(n, (1, 1)), unit(n, (3, 1)), unit(n, (4, 1))])
    x = b.load("x", [unit(n, (0, 1)), unit(n, (3, 1)), unit(n, (2, 2), (4, 1))])
    prod = b.bin("mul", w, x)
    inner = b.sum(4, 0, nu - 1, prod)
    b.sum(3, 0, nc - 1, inner)
    return b.done()


# --------------------------------------------------------------------------- #
# the five workloads at full size, and reduced versions of the same structure
# --------------------------------------------------------------------------- #

def _conv_full() -> Expr:
    e = conv1d(64, 256, 256, 2048, 5, name="cfg5_conv1d")
    e.arg_shapes[0] = [64, 256, 4099]   # 2t+u <= 4098; the stated length
    return e


def _shifted_full() -> Expr:
    return shifted(4096, x_len=20478, name="cfg3_shifted")   # 2 unread tail elements


FULL = {
    "cfg1": lambda: intro(64, 64, 5, name="cfg1_intro"),
    "cfg2": lambda: intro(8192, 8192, 32, name="cfg2_intro_scaled"),
    "cfg3": _shifted_full,
    "cfg4": lambda: nonunimodular(512, name="cfg4_nonunimodular"),
    "cfg5": _conv_full,
}

# Reduced cases with the same structure: small enough for a full oracle run in
# seconds, sized to span several thread-block tiles and leave ragged tails.
REDUCED = {
    "cfg1": lambda: intro(64, 64, 5, name="cfg1_intro"),
    "cfg2": lambda: intro(203, 157, 7, name="cfg2_reduced"),
    "cfg3": lambda: shifted(301, x_len=5 * 300 + 3, name="cfg3_reduced"),
    "cfg4": lambda: nonunimodular(37, name="cfg4_reduced"),
    "cfg5": lambda: conv1d(3, 13, 11, 70, 5, name="cfg5_reduced"),
}

def profile_case(key: str, rows: int) -> Expr:
    """The structure of a full workload with a smaller leading extent: for profiler captures (a few
    launches of a kernel whose tensors still exceed the L2 cache), never a benchmark number."""
    if key == "cfg2":
        return intro(rows, 8192, 32, name=f"cfg2_intro_scaled_rows{rows}")
    if key == "cfg3":
        return shifted(rows, name=f"cfg3_shifted_rows{rows}")
    if key == "cfg4":
        return nonunimodular(rows, name=f"cfg4_nonunimodular_rows{rows}")
    if key == "cfg5":
        e = conv1d(rows, 256, 256, 2048, 5, name=f"cfg5_conv1d_rows{rows}")
        e.arg_shapes[0] = [rows, 256, 4099]
        return e
    raise ValueError("no reduced profile case for " + key)


# value distributions per workload: ("uniform", lo, hi) or ("normal", mean, std)
DIST = {
    "cfg1": ("uniform", -0.5, 0.5),
    "cfg2": ("uniform", -0.5, 0.5),
    "cfg3": ("uniform", -1.0, 1.0),
    "cfg4": ("normal", 0.0, 1.0),
    "cfg5": ("normal", 0.0, 0.1),
}


def make_inputs(e: Expr, dist: Tuple[str, float, float], seed: int = 0
                ) -> Tuple[List[torch.Tensor], torch.Tensor]:
    """Arguments (declaration order) then df ~ N(0, 1); fp32, CPU, contiguous."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    args = []
    for shape in e.arg_shapes:
        if dist[0] == "uniform":
            t = torch.rand(shape, generator=g, dtype=torch.float32) * (dist[2] - dist[1]) + dist[1]
        else:
            t = torch.randn(shape, generator=g, dtype=torch.float32) * dist[2] + dist[1]
        args.append(t.contiguous())
    df = torch.randn(e.out_shape, generator=g, dtype=torch.float32).contiguous()
    return args, df


def workload(key: str, full: bool = False, seed: int = 0):
    e = (FULL if full else REDUCED)[key]()
    args, df = make_inputs(e, DIST[key], seed)
    return e, args, df


# --------------------------------------------------------------------------- #
# the paper's small worked examples (used to pin the oracle and the plans)
# --------------------------------------------------------------------------- #

def ex_square_broadcast(ni: int, nj: int) -> Expr:
    """f_ij = x_i^2  (Sec. 1)."""
    b = Builder("ex_square_broadcast", [ni, nj], 0, ["x"], [[ni]])
    b.powi(b.load("x", [unit(2, (0, 1))]), 2)
    return b.done()


def ex_diag_square(n: int) -> Expr:
    """f_i = x_ii^2  (Sec. 1)."""
    b = Builder("ex_diag_square", [n], 0, ["x"], [[n, n]])
    b.powi(b.load("x", [unit(1, (0, 1)), unit(1, (0, 1))]), 2)
    return b.done()


def ex_exp_shift(ni: int, nj: int) -> Expr:
    """f_ij = exp x_{i+j}  (Sec. 1)."""
    b = Builder("ex_exp_shift", [ni, nj], 0, ["x"], [[ni + nj - 1]])
    b.un("exp", b.load("x", [unit(2, (0, 1), (1, 1))]))
    return b.done()


def ex_sin(n: int) -> Expr:
    """f^1_i = sin x_i  (Sec. 5)."""
    b = Builder("ex_sin", [n], 0, ["x"], [[n]])
    b.un("sin", b.load("x", [unit(1, (0, 1))]))
    return b.done()


def ex_unary(fn: str, n: int) -> Expr:
    """f_i = fn(x_i) for one elementary function (argument sweeps of the function tests)."""
    b = Builder("ex_" + fn, [n], 0, ["x"], [[n]])
    b.un(fn, b.load("x", [unit(1, (0, 1))]))
    return b.done()


def function_sweep(fn: str, n: int = 8192, seed: int = 0):
    """Arguments that exercise an elementary function over its whole useful range: moderate and
    large magnitudes, values next to multiples of pi / 2 and around the switch points of
    piecewise evaluations, tiny values, zeros.  Returns (expr, [x], df)."""
    import math
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    q = n // 8
    parts = [
        (torch.rand(q, generator=g) * 2 - 1) * 10.0,
        torch.randn(q, generator=g) * (30.0 if fn in ("exp", "sinh", "cosh") else 3000.0),
        torch.round(torch.randn(q, generator=g) * 40) * (math.pi / 2) + (torch.rand(q, generator=g) - 0.5) * 1e-3,
        (torch.rand(q, generator=g) * 2 - 1) * 0.5,
        0.25 + (torch.rand(q, generator=g) - 0.5) * 1e-4,
        (torch.rand(q, generator=g) * 2 - 1) * 1e-5,
        torch.randn(q, generator=g) * (80.0 if fn in ("exp", "sinh", "cosh") else 3.0e5),
    ]
    x = torch.cat(parts)
    x = torch.cat([x, torch.zeros(n - x.numel())]).to(torch.float32)
    if fn == "log":
        x = x.abs() + 1e-3
    if fn in ("exp", "sinh", "cosh"):
        x = x.clamp(-85.0, 85.0)
    df = torch.randn(n, generator=g, dtype=torch.float32)
    return ex_unary(fn, n), [x.contiguous()], df.contiguous()


def ex_xy(n: int) -> Expr:
    """f^2_ij = x_i y_ij  (Sec. 5)."""
    b = Builder("ex_xy", [n, n], 0, ["x", "y"], [[n], [n, n]])
    b.bin("mul", b.load("x", [unit(2, (0, 1))]), b.load("y", [unit(2, (0, 1)), unit(2, (1, 1))]))
    return b.done()


def ex_diag_cube(n: int) -> Expr:
    """f^3_i = x_ii^3  (Sec. 5)."""
    b = Builder("ex_diag_cube", [n], 0, ["x"], [[n, n]])
    b.powi(b.load("x", [unit(1, (0, 1)), unit(1, (0, 1))]), 3)
    return b.done()


def ex_matmul(ni: int, nk: int, nj: int) -> Expr:
    """f^4_ij = sum_k x_ik y_kj  (Sec. 5)."""
    b = Builder("ex_matmul", [ni, nj], 1, ["x", "y"], [[ni, nk], [nk, nj]])
    x = b.load("x", [unit(3, (0, 1)), unit(3, (2, 1))])
    y = b.load("y", [unit(3, (2, 1)), unit(3, (1, 1))])
    b.sum(2, 0, nk - 1, b.bin("mul", x, y))
    return b.done()


def ex_matmul_t(ni: int, nj: int, nk: int) -> Expr:
    """f_ij = sum_k x_ik y_jk: the matrix product of Sec. 5 with the second factor stored transposed,
    so that its rows are read along the summation index."""
    b = Builder("ex_matmul_t", [ni, nj], 1, ["x", "y"], [[ni, nk], [nj, nk]])
    x = b.load("x", [unit(3, (0, 1)), unit(3, (2, 1))])
    y = b.load("y", [unit(3, (1, 1)), unit(3, (2, 1))])
    b.sum(2, 0, nk - 1, b.bin("mul", x, y))
    return b.done()


def ex_rowsum_sq(n: int, nk: int) -> Expr:
    """f_j = sum_k (y_jk)^2 + w_k: every output sums along a row of y."""
    b = Builder("ex_rowsum_sq", [n], 1, ["y", "w"], [[n, nk], [nk]])
    y = b.load("y", [unit(2, (0, 1)), unit(2, (1, 1))])
    w = b.load("w", [unit(2, (1, 1))])
    b.sum(1, 0, nk - 1, b.bin("add", b.powi(y, 2), w))
    return b.done()


def ex_guarded_shared_fn(ni: int, nj: int, ns: int, nt: int) -> Expr:
    """f_ij = sum_s (cos x_{i+1} + w_s) tanh(sum_t 0.1 y_{nj-1-j}^2) with x longer than the image of i + 1: the
    gradient of x has elements with no term at both ends, and the function of the inner sum is the same
    for every element of x."""
    b = Builder("ex_guarded_shared_fn", [ni, nj], 2, ["x", "y", "w"], [[nj], [nj], [ns]])
    xi = b.load("x", [[1, 0, 0, 0]], [1])
    ws = b.load("w", [[0, 0, 1, 0]])
    yj = b.load("y", [[0, -1, 0, 0]], [nj - 1])
    inner = b.sum(3, 0, nt - 1, b.bin("mul", b.powi(yj, 2), b.const(0.1)))
    b.sum(2, 0, ns - 1, b.bin("mul", b.bin("add", b.un("cos", xi), ws), b.un("tanh", inner)))
    return b.done()


def ex_exp_flat(n: int, m: int) -> Expr:
    """f^5_ij = exp x_{M i + j}, i in [0, n), j in [0, m)  (Sec. 5)."""
    b = Builder("ex_exp_flat", [n, m], 0, ["x"], [[n * m]])
    b.un("exp", b.load("x", [unit(2, (0, m), (1, 1))]))
    return b.done()


def ex_section6() -> Expr:
    """The example of Sec. 6: a 3x5, b 4x5, c 3x3, d 8 (one unread element), f 3x4."""
    return intro(3, 4, 5, c_cols=3, d_len=8, name="ex_section6")


def ex_strided(n: int, stride: int) -> Expr:
    """f_i = x_{stride*i}^2: odd argument indices have no integer pre-image."""
    b = Builder("ex_strided", [n], 0, ["x"], [[stride * (n - 1) + 1]])
    b.powi(b.load("x", [unit(1, (0, stride))]), 2)
    return b.done()


def ex_strided2(ni: int, nj: int) -> Expr:
    """f_ij = sin x_{2i+4j}: image lattice has index 2."""
    b = Builder("ex_strided2", [ni, nj], 0, ["x"], [[2 * (ni - 1) + 4 * (nj - 1) + 1]])
    b.un("sin", b.load("x", [unit(2, (0, 2), (1, 4))]))
    return b.done()


def ex_lattice2d(ni: int, nj: int) -> Expr:
    """f_ij = cos x_{2i+j, 2j}: square map with determinant 4."""
    b = Builder("ex_lattice2d", [ni, nj], 0, ["x"], [[2 * (ni - 1) + nj, 2 * (nj - 1) + 1]])
    b.un("cos", b.load("x", [unit(2, (0, 2), (1, 1)), unit(2, (1, 2))]))
    return b.done()


def ex_all_ops(n: int) -> Expr:
    """Every elementary function once, with a shared subexpression and a nested sum.

    f_i = sum_k [ log(u_ik^2 + 1.5) / cosh(v_k) + sinh(u_ik) * cos(v_k) ]
          - tanh(u_i0) * sin(u_i0) + exp(-v_1) ** 3 + u_{i0}^(-2 applied to (2+u_i0))
    """
    nk = 3
    b = Builder("ex_all_ops", [n], 1, ["u", "v"], [[n, nk], [nk]])
    u = b.load("u", [unit(2, (0, 1)), unit(2, (1, 1))])
    v = b.load("v", [unit(2, (1, 1))])
    u2 = b.powi(u, 2)
    lg = b.un("log", b.bin("add", u2, b.const(1.5)))
    t1 = b.bin("div", lg, b.un("cosh", v))
    t2 = b.bin("mul", b.un("sinh", u), b.un("cos", v))
    sm = b.sum(1, 0, nk - 1, b.bin("add", t1, t2))
    u0 = b.load("u", [unit(2, (0, 1)), unit(2)])
    t3 = b.bin("mul", b.un("tanh", u0), b.un("sin", u0))
    v1 = b.load("v", [unit(2)], [1])
    t4 = b.powi(b.un("exp", b.un("neg", v1)), 3)
    t5 = b.powi(b.bin("add", b.const(2.0), u0), -2)
    b.bin("add", b.bin("add", b.bin("sub", sm, t3), t4), t5)
    return b.done()

"""Seeded random expressions for the parity tests: random integer affine index maps (strides,
negative coefficients, repeated and constant indices, several index expressions per argument),
random trees of elementary functions, optionally one inner sum (level 3: two sums, one inside
the other, with leaves at every depth).  Data only: nothing here evaluates an expression."""
from __future__ import annotations

from typing import List

import numpy as np

from .expr import Builder, Expr


def random_expression(seed: int, large: int = 0) -> Expr:
    """large = 1, 2: extents at which split summations, then the wide vector shapes and element variables apply;
    large = 3: a sum of up to 40 terms inside a sum of up to 12, medium extents;
    large = 4: one or two sums, the inner one up to 64 terms, up to 2e5 outputs, and the remaining elementary
    functions (log, division, sinh, cosh) with arguments kept inside their domains;
    large = 5: contractions, a product of two index expressions under one or two sums (the product kernels)."""
    if large == 5:
        return _random_contraction(seed)
    rng = np.random.default_rng(seed + 100003 * large)
    n_out = int(rng.integers(1, 4))
    top = [[48, 14, 7], [6000, 400, 48], [3000000, 1800, 150], [3000, 160, 28], [200000, 600, 60]][large]
    out_shape = [int(rng.integers(max(2, top[n_out - 1] // 3) if large else 2, top[n_out - 1] + 1)) for _ in range(n_out)]
    if large == 3:
        n_sum = 2
        sum_lens = [int(rng.integers(1, 13)), int(rng.integers(1, 41))]
    elif large == 4:
        n_sum = int(rng.integers(1, 3))
        sum_lens = [int(rng.integers(1, 9)), int(rng.integers(1, 65))][2 - n_sum:]
    else:
        n_sum = int(rng.integers(0, 2))
        sum_lens = [int(rng.integers(1, 7))] if n_sum else []
    sum_len = sum_lens[0] if n_sum else 0
    n_idx = n_out + n_sum
    ext = out_shape + sum_lens
    n_args = int(rng.integers(1, 4))
    names = ["x", "y", "w"][:n_args]
    ranks = [int(rng.integers(1, 3)) for _ in range(n_args)]

    # leaves: (argument, rows, offset) with every index inside [0, shape)
    leaves = []
    shapes = [[1] * r for r in ranks]

    def make_leaf(inside_sum):
        # arguments stay below 3 M elements: a leaf that would make its argument larger is drawn again
        for _ in range(50):
            saved = [list(sh) for sh in shapes]
            leaf = draw_leaf(inside_sum)
            if int(np.prod(shapes[leaf[0]], dtype=np.int64)) <= 3_000_000:
                return leaf
            for k, sh in enumerate(saved):
                shapes[k][:] = sh
        # a constant index always fits
        p = int(rng.integers(0, n_args))
        return p, [[0] * n_idx for _ in range(ranks[p])], [0] * ranks[p]

    def draw_leaf(inside_sum):
        # inside_sum: False = output indices only, True = all indices, an int = that many leading indices
        n_allowed = n_out if inside_sum is False else n_idx if inside_sum is True else int(inside_sum)
        p = int(rng.integers(0, n_args))
        rows, offs = [], []
        for r in range(ranks[p]):
            row = [0] * n_idx
            for d in range(n_idx):
                if d >= n_allowed:
                    continue
                if rng.random() < 0.55:
                    row[d] = int(rng.choice([1, 1, 1, 2, 3, -1, -2]))
            lo = sum(min(0, c * (ext[d] - 1)) for d, c in enumerate(row))
            hi = sum(max(0, c * (ext[d] - 1)) for d, c in enumerate(row))
            off = -lo + int(rng.integers(0, 3))
            rows.append(row); offs.append(off)
            shapes[p][r] = max(shapes[p][r], hi + off + 1 + int(rng.integers(0, 2)))
        return p, rows, offs

    n_in = int(rng.integers(1, 4)) if n_sum else 0
    n_outside = int(rng.integers(1 if not n_sum else 0, 4))
    inside = [make_leaf(True) for _ in range(n_in)]
    outside = [make_leaf(False) for _ in range(n_outside)]
    middle = [make_leaf(n_out + 1) for _ in range(int(rng.integers(0, 3)))] if large >= 3 and n_sum == 2 else []

    b = Builder(f"random_{large}_{seed}", out_shape, n_sum, names, shapes)
    # the shapes grew while the leaves were drawn
    b.e.arg_shapes = [list(s) for s in shapes]

    def tree(leaf_ids: List[int], n_leaves: int = -1) -> int:
        # level 3 applies functions to index expressions only (n_leaves of the ids), never to a sum: a function of
        # a long cancelling sum is ill-conditioned in fp32 and says nothing about the code under test
        nodes = list(leaf_ids)
        for k in range(len(nodes)):
            if large >= 3 and k >= n_leaves:
                continue
            if large == 4 and rng.random() < 0.35:
                # arguments are drawn from [-1, 1]: 1.5 + x and 2 + x stay positive
                op = str(rng.choice(["log", "recip", "sinh", "cosh", "quot"]))
                if op == "log":
                    nodes[k] = b.un("log", b.bin("add", nodes[k], b.const(1.5)))
                elif op == "recip":
                    nodes[k] = b.bin("div", b.const(1.0), b.bin("add", nodes[k], b.const(2.0)))
                elif op == "quot":
                    nodes[k] = b.bin("div", nodes[k], b.bin("add", b.powi(nodes[k], 2), b.const(1.0)))
                else:
                    nodes[k] = b.un(op, nodes[k])
                continue
            if rng.random() < 0.5:
                op = str(rng.choice(["sin", "cos", "tanh", "exp", "neg", "sq", "cube"]))
                nodes[k] = b.powi(nodes[k], 2) if op == "sq" else b.powi(nodes[k], 3) if op == "cube" else b.un(op, nodes[k])
        while len(nodes) > 1:
            i = int(rng.integers(0, len(nodes) - 1))
            op = str(rng.choice(["add", "mul", "mul", "sub"]))
            nodes[i:i + 2] = [b.bin(op, nodes[i], nodes[i + 1])]
        root = nodes[0]
        if rng.random() < 0.3:
            root = b.bin("mul", root, b.const(float(rng.choice([2.0, -0.5, 3.0]))))
        return root

    parts = [b.load(names[p], rows, offs) for p, rows, offs in outside]
    if n_sum == 2:
        inner = b.sum(n_out + 1, 0, sum_lens[1] - 1, tree([b.load(names[p], rows, offs) for p, rows, offs in inside], len(inside)))
        body = tree([b.load(names[p], rows, offs) for p, rows, offs in middle] + [inner], len(middle))
        parts.append(b.sum(n_out, 0, sum_lens[0] - 1, body))
        tree(parts, len(outside))
        return b.done()
    elif large == 4:
        body = tree([b.load(names[p], rows, offs) for p, rows, offs in inside], len(inside))
        parts.append(b.sum(n_out, 0, sum_len - 1, body))
        tree(parts, len(outside))
        return b.done()
    elif n_sum:
        body = tree([b.load(names[p], rows, offs) for p, rows, offs in inside])
        parts.append(b.sum(n_out, 0, sum_len - 1, body))
    root = tree(parts)
    if rng.random() < 0.3:
        b.un(str(rng.choice(["exp", "tanh", "sin"])), root)
    return b.done()


def _random_contraction(seed: int) -> Expr:
    """f_alpha = sum_{s0[, s1]} x[...] * y[...] with random index maps: every index appears in at least one
    factor, coefficients from {1, 1, 1, 2, -1}; 4e4 .. 4e6 outputs, 8 .. 300 terms each."""
    rng = np.random.default_rng(seed + 100003 * 5)
    n_out = int(rng.integers(2, 4))
    sizes = [[int(rng.integers(100, 800)), int(rng.integers(400, 3000))],
             [int(rng.integers(2, 20)), int(rng.integers(16, 160)), int(rng.integers(200, 1200))]][n_out - 2]
    out_shape = [int(v) for v in rng.permutation(sizes)]
    n_sum = int(rng.integers(1, 3))
    sum_lens = [int(rng.integers(8, 65))] if n_sum == 1 else [int(rng.integers(8, 49)), int(rng.integers(2, 7))]
    n_idx = n_out + n_sum
    ext = out_shape + sum_lens
    ranks = [int(rng.integers(1, 4)), int(rng.integers(1, 4))]
    while True:
        maps = []
        for r in ranks:
            rows = [[0] * n_idx for _ in range(r)]
            for d in range(n_idx):
                if rng.random() < 0.6:
                    rows[int(rng.integers(0, r))][d] = int(rng.choice([1, 1, 1, 2, -1]))
            maps.append(rows)
        used = [any(rows[k][d] for rows in maps for k in range(len(rows))) for d in range(n_idx)]
        sizes_ok = True
        shapes, offsets = [], []
        for rows in maps:
            shape, offs = [], []
            for row in rows:
                lo = sum(min(0, c * (ext[d] - 1)) for d, c in enumerate(row))
                hi = sum(max(0, c * (ext[d] - 1)) for d, c in enumerate(row))
                shift = int(rng.integers(0, 2))
                offs.append(-lo + shift)
                shape.append(hi - lo + 1 + shift + int(rng.integers(0, 3)))
            shapes.append(shape); offsets.append(offs)
            if int(np.prod(shape, dtype=np.int64)) > 3_000_000:
                sizes_ok = False
        if all(used) and sizes_ok:
            break
    b = Builder(f"random_5_{seed}", out_shape, n_sum, ["x", "y"], shapes)
    prod = b.bin("mul", b.load("x", maps[0], offsets[0]), b.load("y", maps[1], offsets[1]))
    for k in range(n_sum - 1, -1, -1):
        prod = b.sum(n_out + k, 0, sum_lens[k] - 1, prod)
    return b.done()

"""Neutral description of an element-wise defined tensor expression.

This module holds data only: shapes, integer index matrices, offsets and a node
list.  It performs none of the method's arithmetic (no evaluation, no
differentiation, no index inversion).  Both the CPU oracle's wrapper and the
CUDA library's binding read these plain fields and marshal them into their own
C structures; neither imports the other.

Model (Sec. 5.1, Sec. 5.2 of the paper): the output element ``f[alpha]`` is a
scalar function of argument elements ``x^p[A alpha_hat + o]`` where
``alpha_hat = [alpha, k_1, ..., k_S]`` is the output multi-index extended by the
indices of the sums that occur in the expression.  Indices are zero-based and
tensors are row-major.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence

OPS = ("const", "load", "neg", "add", "sub", "mul", "div", "powi", "exp", "log",
       "sin", "cos", "tanh", "sinh", "cosh", "sum")


@dataclass
class Access:
    """One index expression of one argument: ``x^arg[A @ alpha_hat + offset]``."""
    arg: int
    A: List[List[int]]          # rank(arg) x n_idx, n_idx = len(out_shape) + n_sum_idx
    offset: List[int]           # rank(arg)


@dataclass
class Node:
    op: str
    in0: int = -1
    in1: int = -1
    access: int = -1            # op == "load"
    ipow: int = 0               # op == "powi": literal integer exponent
    sum_idx: int = -1           # op == "sum": position of its index inside alpha_hat
    sum_lo: int = 0             # inclusive
    sum_hi: int = 0             # inclusive
    imm: float = 0.0            # op == "const"


@dataclass
class Expr:
    name: str
    out_shape: List[int]
    n_sum_idx: int
    arg_names: List[str]
    arg_shapes: List[List[int]]
    accesses: List[Access] = field(default_factory=list)
    nodes: List[Node] = field(default_factory=list)   # topological order, root last

    @property
    def n_idx(self) -> int:
        return len(self.out_shape) + self.n_sum_idx


class Builder:
    """Small helper that appends nodes in topological order and returns their ids."""

    def __init__(self, name: str, out_shape: Sequence[int], n_sum_idx: int,
                 arg_names: Sequence[str], arg_shapes: Sequence[Sequence[int]]):
        self.e = Expr(name, list(out_shape), n_sum_idx, list(arg_names),
                      [list(s) for s in arg_shapes])

    def _push(self, node: Node) -> int:
        self.e.nodes.append(node)
        return len(self.e.nodes) - 1

    def load(self, arg: str, rows: Sequence[Sequence[int]], offset: Sequence[int] | None = None) -> int:
        p = self.e.arg_names.index(arg)
        rows = [list(r) for r in rows]
        assert len(rows) == len(self.e.arg_shapes[p])
        assert all(len(r) == self.e.n_idx for r in rows)
        offset = [0] * len(rows) if offset is None else list(offset)
        acc = Access(p, rows, offset)
        for q, other in enumerate(self.e.accesses):
            if other == acc:
                break
        else:
            self.e.accesses.append(acc)
            q = len(self.e.accesses) - 1
        return self._push(Node("load", access=q))

    def const(self, v: float) -> int:
        return self._push(Node("const", imm=float(v)))

    def un(self, op: str, a: int) -> int:
        assert op in ("neg", "exp", "log", "sin", "cos", "tanh", "sinh", "cosh")
        return self._push(Node(op, in0=a))

    def bin(self, op: str, a: int, b: int) -> int:
        assert op in ("add", "sub", "mul", "div")
        return self._push(Node(op, in0=a, in1=b))

    def powi(self, a: int, n: int) -> int:
        return self._push(Node("powi", in0=a, ipow=int(n)))

    def sum(self, sum_idx: int, lo: int, hi: int, body: int) -> int:
        assert len(self.e.out_shape) <= sum_idx < self.e.n_idx
        return self._push(Node("sum", in0=body, sum_idx=sum_idx, sum_lo=lo, sum_hi=hi))

    def done(self) -> Expr:
        return self.e


def unit(n_idx: int, *pairs: Sequence[int]) -> List[int]:
    """Row of an index matrix: ``unit(3, (0, 2), (1, 3))`` is ``2*idx0 + 3*idx1``."""
    row = [0] * n_idx
    for pos, coef in pairs:
        row[pos] += coef
    return row

"""ctypes wrapper around the float64 CPU oracle (``tad_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing in the product imports this; it shares no
code with the CUDA library.  Inputs are the fp32 tensors the GPU path gets,
widened to float64 here.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tad_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

_OPCODE = {"const": 1, "load": 2, "neg": 3, "add": 4, "sub": 5, "mul": 6, "div": 7, "powi": 8,
           "exp": 9, "log": 10, "sin": 11, "cos": 12, "tanh": 13, "sinh": 14, "cosh": 15, "sum": 16}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Node(C.Structure):
    _fields_ = [("op", C.c_int32), ("in0", C.c_int32), ("in1", C.c_int32), ("access", C.c_int32),
                ("ipow", C.c_int32), ("sum_idx", C.c_int32), ("sum_lo", C.c_int64),
                ("sum_hi", C.c_int64), ("imm", C.c_double)]


class _Access(C.Structure):
    _fields_ = [("arg", C.c_int32), ("rank", C.c_int32),
                ("A", C.POINTER(C.c_int64)), ("off", C.POINTER(C.c_int64))]


class _Expr(C.Structure):
    _fields_ = [("n_out_dims", C.c_int32), ("out_shape", C.POINTER(C.c_int64)),
                ("n_sum_idx", C.c_int32), ("n_args", C.c_int32),
                ("arg_rank", C.POINTER(C.c_int32)), ("arg_shape", C.POINTER(C.POINTER(C.c_int64))),
                ("n_access", C.c_int32), ("access", C.POINTER(_Access)),
                ("n_nodes", C.c_int32), ("nodes", C.POINTER(_Node))]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        dpp = C.POINTER(C.POINTER(C.c_double))
        i64p = C.POINTER(C.c_int64)
        _lib.oracle_forward.argtypes = [C.POINTER(_Expr), dpp, i64p, i64p,
                                        C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_int]
        _lib.oracle_backward.argtypes = [C.POINTER(_Expr), dpp, C.POINTER(C.c_double), i64p, i64p,
                                         dpp, dpp, C.c_int]
        _lib.oracle_counts.argtypes = [C.POINTER(_Expr), C.c_int, i64p, i64p, i64p]
        _lib.oracle_max_threads.restype = C.c_int
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _i64(values) -> "C.Array":
    values = [int(v) for v in values]
    return (C.c_int64 * max(1, len(values)))(*values)


class Oracle:
    """Holds the marshalled expression; keeps every ctypes buffer alive."""

    def __init__(self, expr):
        self.expr = expr
        self._keep = []
        e = _Expr()
        e.n_out_dims = len(expr.out_shape)
        shp = _i64(expr.out_shape); self._keep.append(shp)
        e.out_shape = C.cast(shp, C.POINTER(C.c_int64))
        e.n_sum_idx = expr.n_sum_idx
        e.n_args = len(expr.arg_shapes)
        ranks = (C.c_int32 * e.n_args)(*[len(s) for s in expr.arg_shapes]); self._keep.append(ranks)
        e.arg_rank = C.cast(ranks, C.POINTER(C.c_int32))
        shapes = (C.POINTER(C.c_int64) * e.n_args)()
        for p, s in enumerate(expr.arg_shapes):
            buf = _i64(s); self._keep.append(buf)
            shapes[p] = C.cast(buf, C.POINTER(C.c_int64))
        self._keep.append(shapes)
        e.arg_shape = C.cast(shapes, C.POINTER(C.POINTER(C.c_int64)))
        acc = (_Access * max(1, len(expr.accesses)))()
        for q, a in enumerate(expr.accesses):
            flat = _i64([v for row in a.A for v in row]); off = _i64(a.offset)
            self._keep += [flat, off]
            acc[q].arg = a.arg
            acc[q].rank = len(a.A)
            acc[q].A = C.cast(flat, C.POINTER(C.c_int64))
            acc[q].off = C.cast(off, C.POINTER(C.c_int64))
        self._keep.append(acc)
        e.n_access = len(expr.accesses)
        e.access = C.cast(acc, C.POINTER(_Access))
        nodes = (_Node * len(expr.nodes))()
        for i, n in enumerate(expr.nodes):
            nodes[i].op = _OPCODE[n.op]
            nodes[i].in0, nodes[i].in1 = n.in0, n.in1
            nodes[i].access, nodes[i].ipow = n.access, n.ipow
            nodes[i].sum_idx, nodes[i].sum_lo, nodes[i].sum_hi = n.sum_idx, n.sum_lo, n.sum_hi
            nodes[i].imm = n.imm
        self._keep.append(nodes)
        e.n_nodes = len(expr.nodes)
        e.nodes = C.cast(nodes, C.POINTER(_Node))
        self._e = e

    # ------------------------------------------------------------------ #
    def _box(self, lo, hi):
        nd = len(self.expr.out_shape)
        lo = [0] * nd if lo is None else list(lo)
        hi = list(self.expr.out_shape) if hi is None else list(hi)
        return _i64(lo), _i64(hi)

    @staticmethod
    def _f64(arrays: Sequence) -> List[np.ndarray]:
        out = []
        for a in arrays:
            a = a.detach().cpu().numpy() if hasattr(a, "detach") else np.asarray(a)
            out.append(np.ascontiguousarray(a, dtype=np.float64))
        return out

    def _ptrs(self, arrays: Sequence[Optional[np.ndarray]]):
        pp = (C.POINTER(C.c_double) * max(1, len(arrays)))()
        for i, a in enumerate(arrays):
            pp[i] = a.ctypes.data_as(C.POINTER(C.c_double)) if a is not None else None
        return pp

    def forward(self, args, lo=None, hi=None, nthreads: int = 1):
        """Returns (f, f_abs) as float64 arrays of the output shape (sub-box written, rest 0)."""
        a64 = self._f64(args)
        for a, s in zip(a64, self.expr.arg_shapes):
            assert list(a.shape) == list(s), (a.shape, s)
        f = np.zeros(self.expr.out_shape, dtype=np.float64)
        fabs = np.zeros(self.expr.out_shape, dtype=np.float64)
        blo, bhi = self._box(lo, hi)
        rc = _load().oracle_forward(C.byref(self._e), self._ptrs(a64), blo, bhi,
                                    f.ctypes.data_as(C.POINTER(C.c_double)),
                                    fabs.ctypes.data_as(C.POINTER(C.c_double)), nthreads)
        if rc:
            raise RuntimeError(f"oracle_forward failed with status {rc}")
        return f, fabs

    def backward(self, args, df, lo=None, hi=None, wanted=None, nthreads: int = 1):
        """Returns (dx, t_abs): per argument float64 gradient and sum of |terms| (None if not wanted)."""
        a64 = self._f64(args)
        df64 = self._f64([df])[0]
        assert list(df64.shape) == list(self.expr.out_shape)
        n = len(a64)
        wanted = [True] * n if wanted is None else list(wanted)
        dx = [np.zeros(s, dtype=np.float64) if w else None for s, w in zip(self.expr.arg_shapes, wanted)]
        tb = [np.zeros(s, dtype=np.float64) if w else None for s, w in zip(self.expr.arg_shapes, wanted)]
        blo, bhi = self._box(lo, hi)
        rc = _load().oracle_backward(C.byref(self._e), self._ptrs(a64),
                                     df64.ctypes.data_as(C.POINTER(C.c_double)), blo, bhi,
                                     self._ptrs(dx), self._ptrs(tb), nthreads)
        if rc:
            raise RuntimeError(f"oracle_backward failed with status {rc}")
        return dx, tb

    def counts(self, access: int, lo=None, hi=None) -> np.ndarray:
        """Term count per element of the argument that index expression `access` reads."""
        shape = self.expr.arg_shapes[self.expr.accesses[access].arg]
        cnt = np.zeros(shape, dtype=np.int64)
        blo, bhi = self._box(lo, hi)
        rc = _load().oracle_counts(C.byref(self._e), access, blo, bhi,
                                   cnt.ctypes.data_as(C.POINTER(C.c_int64)))
        if rc:
            raise RuntimeError(f"oracle_counts failed with status {rc}")
        return cnt

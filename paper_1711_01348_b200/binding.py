"""Thin ctypes binding of libtad.so: argument marshalling only.

Every step of the path (compile-time integer algebra, code generation, forward and backward
kernels) runs inside the library.  There is no fallback: if the library cannot be loaded the
import fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libtad.so")

OPCODE = {"const": 0, "load": 1, "neg": 2, "add": 3, "sub": 4, "mul": 5, "div": 6, "powi": 7,
          "exp": 8, "log": 9, "sin": 10, "cos": 11, "tanh": 12, "sinh": 13, "cosh": 14, "sum": 15}

STATUS = {0: "TAD_OK", 1: "TAD_ERR_INVALID_ARG", 2: "TAD_ERR_BAD_EXPR", 3: "TAD_ERR_OUT_OF_RANGE",
          4: "TAD_ERR_OVERFLOW", 5: "TAD_ERR_UNSUPPORTED", 6: "TAD_ERR_WORKSPACE", 7: "TAD_ERR_CUDA",
          8: "TAD_ERR_NOMEM"}

MAX_IDX, MAX_RANK, MAX_KAPPA = 8, 4, 4

EXPORTS = ["tad_compile", "tad_destroy", "tad_workspace_bytes", "tad_forward", "tad_backward",
           "tad_backward_stage", "tad_backward_arg", "tad_plan_num_stages", "tad_backward_noalloc",
           "tad_staging_bytes", "tad_step_host", "tad_last_error", "tad_debug_status",
           "tad_plan_access_info", "tad_plan_bound_row", "tad_plan_enumerate", "tad_plan_kernel_stats",
           "tad_plan_disassemble", "tad_plan_print", "tad_extended_euclid", "tad_smith_normal_form", "tad_fourier_motzkin",
           "tad_measure_fp32_rate"]


class TadError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{STATUS.get(status, status)}: {text}")
        self.status = status
        self.code = STATUS.get(status, str(status))


class _Access(C.Structure):
    _fields_ = [("arg", C.c_int32), ("A", C.POINTER(C.c_int64)), ("offset", C.POINTER(C.c_int64))]


class _Node(C.Structure):
    _fields_ = [("op", C.c_int32), ("in0", C.c_int32), ("in1", C.c_int32), ("access", C.c_int32),
                ("ipow", C.c_int32), ("sum_idx", C.c_int32), ("sum_lo", C.c_int64), ("sum_hi", C.c_int64),
                ("imm", C.c_double)]


class _Expr(C.Structure):
    _fields_ = [("n_out_dims", C.c_int32), ("out_shape", C.POINTER(C.c_int64)), ("n_sum_idx", C.c_int32),
                ("n_args", C.c_int32), ("arg_rank", C.POINTER(C.c_int32)),
                ("arg_shape", C.POINTER(C.POINTER(C.c_int64))),
                ("n_access", C.c_int32), ("access", C.POINTER(_Access)),
                ("n_nodes", C.c_int32), ("nodes", C.POINTER(_Node))]


class _Options(C.Structure):
    _fields_ = [("debug_bounds", C.c_int32), ("saved_forward", C.c_int32), ("reserved", C.c_int32 * 6)]


class AccessInfo(C.Structure):
    _fields_ = [("arg", C.c_int32), ("rank", C.c_int32), ("n_idx", C.c_int32), ("idx_pos", C.c_int32 * MAX_IDX),
                ("R", C.c_int32), ("kappa", C.c_int32),
                ("A", C.c_int64 * (MAX_RANK * MAX_IDX)), ("offset", C.c_int64 * MAX_RANK),
                ("S", C.c_int64 * MAX_RANK), ("U", C.c_int64 * (MAX_RANK * MAX_RANK)),
                ("V", C.c_int64 * (MAX_IDX * MAX_IDX)),
                ("box_lo", C.c_int64 * MAX_IDX), ("box_hi", C.c_int64 * MAX_IDX),
                ("n_lower", C.c_int32 * MAX_KAPPA), ("n_upper", C.c_int32 * MAX_KAPPA),
                ("masked", C.c_int32), ("lane_var", C.c_int32)]


class KernelStats(C.Structure):
    _fields_ = [("outputs", C.c_int64), ("terms", C.c_int64),
                ("alg_bytes", C.c_double), ("alg_flops", C.c_double), ("alg_transcendentals", C.c_double),
                ("bytecode_words", C.c_int32), ("n_launches", C.c_int32)]


def _load() -> C.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with paper_1711_01348_b200/build.py "
                          "(there is no fallback path)")
    lib = C.CDLL(_LIB_PATH)
    vp, i64p, i32p = C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int32)
    lib.tad_compile.argtypes = [C.POINTER(_Expr), C.POINTER(_Options), C.POINTER(vp)]
    lib.tad_destroy.argtypes = [vp]; lib.tad_destroy.restype = None
    lib.tad_workspace_bytes.argtypes = [vp]; lib.tad_workspace_bytes.restype = C.c_size_t
    lib.tad_staging_bytes.argtypes = [vp]; lib.tad_staging_bytes.restype = C.c_size_t
    lib.tad_forward.argtypes = [vp, C.POINTER(vp), vp, vp]
    lib.tad_backward.argtypes = [vp, C.POINTER(vp), vp, C.POINTER(vp), vp, C.c_size_t, vp]
    lib.tad_backward_stage.argtypes = [vp, C.POINTER(vp), vp, vp, C.c_size_t, vp]
    lib.tad_backward_arg.argtypes = [vp, C.POINTER(vp), vp, C.c_int32, vp, vp, C.c_size_t, vp]
    lib.tad_backward_noalloc.argtypes = [vp, C.POINTER(vp), vp, C.POINTER(vp), vp]
    lib.tad_plan_num_stages.argtypes = [vp]; lib.tad_plan_num_stages.restype = C.c_int32
    lib.tad_step_host.argtypes = [vp, C.POINTER(vp), vp, vp, C.POINTER(vp), vp, C.c_size_t, vp]
    lib.tad_last_error.restype = C.c_char_p
    lib.tad_debug_status.argtypes = [vp, vp, vp]
    lib.tad_plan_access_info.argtypes = [vp, C.c_int32, C.POINTER(AccessInfo)]
    lib.tad_plan_bound_row.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, i64p, i64p, i64p, i64p]
    lib.tad_plan_enumerate.argtypes = [vp, C.c_int32, i64p, i64p, C.c_size_t, C.POINTER(C.c_size_t)]
    lib.tad_plan_kernel_stats.argtypes = [vp, C.c_int32, C.POINTER(KernelStats)]
    lib.tad_plan_disassemble.argtypes = [vp, C.c_int32, C.c_char_p, C.c_size_t]
    lib.tad_plan_disassemble.restype = C.c_size_t
    lib.tad_plan_print.argtypes = [vp, C.c_int32, C.POINTER(C.c_char_p), C.POINTER(C.c_char_p), C.c_char_p, C.c_size_t]
    lib.tad_plan_print.restype = C.c_size_t
    lib.tad_extended_euclid.argtypes = [C.c_int64, C.c_int64, i64p, i64p, i64p]
    lib.tad_smith_normal_form.argtypes = [i64p, C.c_int32, C.c_int32, i64p, i64p, i64p, i32p]
    lib.tad_fourier_motzkin.argtypes = [i64p, C.c_int32, C.c_int32, C.c_int32, i32p, i32p,
                                        i64p, i64p, i64p, i64p, i64p, i64p, i32p, i64p]
    return lib


lib = _load()


def _check(status: int) -> None:
    if status != 0:
        raise TadError(status, (lib.tad_last_error() or b"").decode())


def _i64(values) -> "C.Array":
    values = [int(v) for v in values]
    return (C.c_int64 * max(1, len(values)))(*values)


class Plan:
    """Owns a tad_plan.  `expr` is any object with the fields of workloads.expr.Expr."""

    def __init__(self, expr, debug_bounds: bool = False, saved_forward: bool = False):
        keep = []
        e = _Expr()
        e.n_out_dims = len(expr.out_shape)
        shp = _i64(expr.out_shape); keep.append(shp)
        e.out_shape = C.cast(shp, C.POINTER(C.c_int64))
        e.n_sum_idx = expr.n_sum_idx
        e.n_args = len(expr.arg_shapes)
        ranks = (C.c_int32 * max(1, e.n_args))(*[len(s) for s in expr.arg_shapes]); keep.append(ranks)
        e.arg_rank = C.cast(ranks, C.POINTER(C.c_int32))
        shapes = (C.POINTER(C.c_int64) * max(1, e.n_args))()
        for p, s in enumerate(expr.arg_shapes):
            b = _i64(s); keep.append(b)
            shapes[p] = C.cast(b, C.POINTER(C.c_int64))
        keep.append(shapes)
        e.arg_shape = C.cast(shapes, C.POINTER(C.POINTER(C.c_int64)))
        acc = (_Access * max(1, len(expr.accesses)))()
        for q, a in enumerate(expr.accesses):
            flat = _i64([v for row in a.A for v in row]); off = _i64(a.offset)
            keep += [flat, off]
            acc[q].arg = a.arg
            acc[q].A = C.cast(flat, C.POINTER(C.c_int64))
            acc[q].offset = C.cast(off, C.POINTER(C.c_int64))
        keep.append(acc)
        e.n_access = len(expr.accesses)
        e.access = C.cast(acc, C.POINTER(_Access))
        nodes = (_Node * max(1, len(expr.nodes)))()
        for i, n in enumerate(expr.nodes):
            nodes[i].op = OPCODE[n.op]
            nodes[i].in0, nodes[i].in1 = n.in0, n.in1
            nodes[i].access, nodes[i].ipow = n.access, n.ipow
            nodes[i].sum_idx, nodes[i].sum_lo, nodes[i].sum_hi = n.sum_idx, n.sum_lo, n.sum_hi
            nodes[i].imm = n.imm
        keep.append(nodes)
        e.n_nodes = len(expr.nodes)
        e.nodes = C.cast(nodes, C.POINTER(_Node))
        opt = _Options()
        opt.debug_bounds = 1 if debug_bounds else 0
        opt.saved_forward = 1 if saved_forward else 0
        self.saved_forward = bool(saved_forward)
        handle = C.c_void_p()
        _check(lib.tad_compile(C.byref(e), C.byref(opt), C.byref(handle)))
        self._h = handle
        self.expr = expr
        self.n_args = e.n_args

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            lib.tad_destroy(h)

    # ---- device entry points (pointers are integers, e.g. torch.Tensor.data_ptr()) ----
    @staticmethod
    def _ptr_array(ptrs: Sequence[Optional[int]]):
        arr = (C.c_void_p * max(1, len(ptrs)))()
        for i, p in enumerate(ptrs):
            arr[i] = p if p else None
        return arr

    def workspace_bytes(self) -> int:
        return int(lib.tad_workspace_bytes(self._h))

    def staging_bytes(self) -> int:
        return int(lib.tad_staging_bytes(self._h))

    def forward(self, arg_ptrs: Sequence[int], f_ptr: int, stream: int = 0,
                workspace_ptr: int = 0, workspace_bytes: int = 0) -> None:
        _check(lib.tad_forward(self._h, self._ptr_array(arg_ptrs), f_ptr, workspace_ptr or None, workspace_bytes,
                               stream or None))

    def backward(self, arg_ptrs: Sequence[int], df_ptr: int, darg_ptrs: Sequence[Optional[int]],
                 workspace_ptr: int = 0, workspace_bytes: int = 0, stream: int = 0) -> None:
        _check(lib.tad_backward(self._h, self._ptr_array(arg_ptrs), df_ptr, self._ptr_array(darg_ptrs),
                                workspace_ptr or None, workspace_bytes, stream or None))

    def backward_stage(self, arg_ptrs, df_ptr, workspace_ptr=0, workspace_bytes=0, stream=0) -> None:
        _check(lib.tad_backward_stage(self._h, self._ptr_array(arg_ptrs), df_ptr,
                                      workspace_ptr or None, workspace_bytes, stream or None))

    def backward_arg(self, arg_ptrs, df_ptr, arg: int, darg_ptr: int, workspace_ptr=0, workspace_bytes=0,
                     stream=0) -> None:
        _check(lib.tad_backward_arg(self._h, self._ptr_array(arg_ptrs), df_ptr, arg, darg_ptr,
                                    workspace_ptr or None, workspace_bytes, stream or None))

    def backward_noalloc(self, arg_ptrs, df_ptr, darg_ptrs, stream: int = 0) -> None:
        """tad_backward with the library's built-in scratch array instead of a caller workspace."""
        _check(lib.tad_backward_noalloc(self._h, self._ptr_array(arg_ptrs), df_ptr,
                                        self._ptr_array(darg_ptrs), stream or None))

    def num_stages(self) -> int:
        return int(lib.tad_plan_num_stages(self._h))

    def step_host(self, h_arg_ptrs, h_df_ptr, h_f_ptr, h_darg_ptrs, staging_ptr, staging_bytes, stream=0) -> None:
        _check(lib.tad_step_host(self._h, self._ptr_array(h_arg_ptrs), h_df_ptr, h_f_ptr or None,
                                 self._ptr_array(h_darg_ptrs), staging_ptr, staging_bytes, stream or None))

    def debug_status(self, workspace_ptr: int, stream: int = 0) -> None:
        _check(lib.tad_debug_status(self._h, workspace_ptr or None, stream or None))

    # ---- introspection (host only) ----
    def access_info(self, q: int) -> AccessInfo:
        info = AccessInfo()
        _check(lib.tad_plan_access_info(self._h, q, C.byref(info)))
        return info

    def bound_rows(self, q: int, loop: int, upper: bool):
        info = self.access_info(q)
        n = (info.n_upper if upper else info.n_lower)[loop]
        rows = []
        for r in range(n):
            den, c0 = C.c_int64(), C.c_int64()
            cx = (C.c_int64 * MAX_RANK)(); cz = (C.c_int64 * MAX_KAPPA)()
            _check(lib.tad_plan_bound_row(self._h, q, loop, int(upper), r, C.byref(den), C.byref(c0), cx, cz))
            rows.append((den.value, c0.value, list(cx)[:info.R], list(cz)[:loop]))
        return rows

    def enumerate(self, q: int, beta: Sequence[int], cap: int = 0) -> tuple:
        """Returns (count, list of alpha_hat tuples) for one argument element."""
        b = _i64(beta)
        n_idx = self.access_info(q).n_idx
        count = C.c_size_t()
        if cap <= 0:
            _check(lib.tad_plan_enumerate(self._h, q, b, None, 0, C.byref(count)))
            return count.value, []
        buf = (C.c_int64 * (cap * n_idx))()
        _check(lib.tad_plan_enumerate(self._h, q, b, buf, cap, C.byref(count)))
        got = min(cap, count.value)
        return count.value, [tuple(buf[i * n_idx + d] for d in range(n_idx)) for i in range(got)]

    def count(self, q: int, beta: Sequence[int]) -> int:
        return self.enumerate(q, beta, 0)[0]

    def kernel_stats(self, which: int) -> KernelStats:
        s = KernelStats()
        _check(lib.tad_plan_kernel_stats(self._h, which, C.byref(s)))
        return s

    def disassemble(self, which: int) -> str:
        n = lib.tad_plan_disassemble(self._h, which, None, 0)
        buf = C.create_string_buffer(n)
        lib.tad_plan_disassemble(self._h, which, buf, n)
        return buf.value.decode()

    def print(self, which: int, arg_names=None, idx_names=None) -> str:
        """tad_plan_print: the expression (which = -1) or the derivative through index expression `which`."""
        def strings(names):
            if names is None:
                return None
            return (C.c_char_p * len(names))(*[n.encode() for n in names])
        a, i = strings(arg_names), strings(idx_names)
        n = lib.tad_plan_print(self._h, which, a, i, None, 0)
        if n == 0:
            return ""
        buf = C.create_string_buffer(n)
        lib.tad_plan_print(self._h, which, a, i, buf, n)
        return buf.value.decode()


# ---- host-only pieces of the integer algebra (for tests) ----

def measure_fp32_rate(stream: int = 0) -> float:
    """TFLOP/s of FP32 multiply-adds from registers on the current device (tad_measure_fp32_rate)."""
    out = C.c_double(0.0)
    _check(lib.tad_measure_fp32_rate(stream or None, C.byref(out)))
    return out.value


def extended_euclid(a: int, b: int):
    g, x, y = C.c_int64(), C.c_int64(), C.c_int64()
    _check(lib.tad_extended_euclid(a, b, C.byref(g), C.byref(x), C.byref(y)))
    return g.value, x.value, y.value


def smith_normal_form(A: List[List[int]]):
    n, m = len(A), len(A[0])
    flat = _i64([v for r in A for v in r])
    S = (C.c_int64 * (n * m))(); U = (C.c_int64 * (n * n))(); V = (C.c_int64 * (m * m))()
    rank = C.c_int32()
    _check(lib.tad_smith_normal_form(flat, n, m, S, U, V, C.byref(rank)))
    mat = lambda buf, r, c: [[buf[i * c + j] for j in range(c)] for i in range(r)]
    return mat(S, n, m), mat(U, n, n), mat(V, m, m), rank.value


def fourier_motzkin(A: List[List[int]], cap_rows: int = 64):
    """Per variable k: (lower, upper) lists of (den, b-coefficients, z-coefficients); and F."""
    n, m = len(A), len(A[0])
    flat = _i64([v for r in A for v in r])
    nl = (C.c_int32 * m)(); nu = (C.c_int32 * m)()
    Ln = (C.c_int64 * (m * cap_rows * n))(); Lh = (C.c_int64 * (m * cap_rows * m))(); Ld = (C.c_int64 * (m * cap_rows))()
    Hn = (C.c_int64 * (m * cap_rows * n))(); Hh = (C.c_int64 * (m * cap_rows * m))(); Hd = (C.c_int64 * (m * cap_rows))()
    nf = C.c_int32(); F = (C.c_int64 * (cap_rows * n))()
    _check(lib.tad_fourier_motzkin(flat, n, m, cap_rows, nl, nu, Ln, Lh, Ld, Hn, Hh, Hd, C.byref(nf), F))
    out = []
    for k in range(m):
        def rows(cnt, num, hat, den):
            res = []
            for i in range(cnt):
                row = k * cap_rows + i
                res.append((den[row], [num[row * n + j] for j in range(n)], [hat[row * m + j] for j in range(m)]))
            return res
        out.append((rows(nl[k], Ln, Lh, Ld), rows(nu[k], Hn, Hh, Hd)))
    feas = [[F[i * n + j] for j in range(n)] for i in range(nf.value)]
    return out, feas

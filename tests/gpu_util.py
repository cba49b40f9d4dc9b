"""Helpers for the GPU parity tests: run the CUDA library through its C ABI on torch-allocated
device buffers and compare with the float64 oracle under the stated tolerance."""
from __future__ import annotations

import numpy as np
import torch

from oracle.oracle import Oracle
from paper_1711_01348_b200 import Plan

RTOL_TERMS = 1e-4      # |gpu - oracle| <= 1e-4 * (sum of |terms| of the element) + 1e-6
ATOL = 1e-6


class GpuRun:
    def __init__(self, expr, args, df, debug_bounds=False, saved_forward=False):
        self.expr = expr
        self.saved_forward = saved_forward
        self.plan = Plan(expr, debug_bounds=debug_bounds, saved_forward=saved_forward)
        dev = torch.device("cuda:0")
        self.args = [a.to(dev).contiguous() for a in args]
        self.df = df.to(dev).contiguous()
        self.f = torch.full(list(expr.out_shape), float("nan"), dtype=torch.float32, device=dev)
        self.dargs = [torch.full(list(s), float("nan"), dtype=torch.float32, device=dev) for s in expr.arg_shapes]
        nbytes = max(256, self.plan.workspace_bytes())
        self.ws = torch.zeros(nbytes, dtype=torch.uint8, device=dev)

    def forward(self):
        stream = torch.cuda.current_stream().cuda_stream
        self.plan.forward([a.data_ptr() for a in self.args], self.f.data_ptr(), stream, self.ws.data_ptr(), self.ws.numel())
        torch.cuda.synchronize()
        return self.f.cpu().numpy()

    def backward(self, wanted=None):
        stream = torch.cuda.current_stream().cuda_stream
        wanted = [True] * len(self.args) if wanted is None else wanted
        # a plan compiled with saved_forward reads the forward output (run forward() first)
        extra = [self.f.data_ptr()] if self.saved_forward else []
        self.plan.backward([a.data_ptr() for a in self.args] + extra, self.df.data_ptr(),
                           [d.data_ptr() if w else 0 for d, w in zip(self.dargs, wanted)],
                           self.ws.data_ptr(), self.ws.numel(), stream)
        torch.cuda.synchronize()
        return [d.cpu().numpy() if w else None for d, w in zip(self.dargs, wanted)]


def assert_close(got, want, scale, what="", mask=None):
    """mask: compare only the elements where it is True (the others are checked to be finite)."""
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - want)
    tol = RTOL_TERMS * scale + ATOL
    bad = ~(err <= tol)      # also catches NaN
    if mask is not None:
        assert np.all(np.isfinite(got[~mask])), f"{what}: non-finite value"
        bad &= mask
    if bad.any():
        idx = np.unravel_index(np.argmax(np.where(bad, err - tol, -np.inf)), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; worst at {idx}: "
                             f"gpu={got[idx]!r} oracle={want[idx]!r} tol={tol[idx]!r}")


def check_against_oracle(expr, args, df, nthreads=1, debug_bounds=False, saved_forward=False, oracle_results=None, masks=None):
    """oracle_results: (f, |f| scale, gradients, term scales) if the caller has them already;
    masks: per tensor (f first, then the gradients), the elements to compare."""
    run = GpuRun(expr, args, df, debug_bounds=debug_bounds, saved_forward=saved_forward)
    if oracle_results is None:
        orc = Oracle(expr)
        f_o, fabs_o = orc.forward(args, nthreads=nthreads)
        dx_o, t_o = orc.backward(args, df, nthreads=nthreads)
    else:
        f_o, fabs_o, dx_o, t_o = oracle_results
    assert_close(run.forward(), f_o, fabs_o, f"{expr.name} forward", None if masks is None else masks[0])
    dx_g = run.backward()
    for p, name in enumerate(expr.arg_names):
        assert_close(dx_g[p], dx_o[p], t_o[p], f"{expr.name} d{name}", None if masks is None else masks[1 + p])
        # elements with an empty Gamma are exactly zero
        assert np.all(dx_g[p][t_o[p] == 0] == 0.0), f"{expr.name} d{name}: non-zero where Gamma is empty"
    if debug_bounds:
        run.plan.debug_status(run.ws.data_ptr())
    return run

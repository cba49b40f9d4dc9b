"""Parity at the full sizes of the five workloads, in the launch configuration the benchmark
times.  Where a full oracle run takes too long the oracle is run on a sub-box of the output
index space and only the gradient elements whose whole Gamma lies in that sub-box are compared
(which ones those are follows from the index expressions by inspection, stated per case)."""
import numpy as np
import pytest

from oracle.oracle import Oracle, max_threads
from workloads import configs as W

pytestmark = pytest.mark.gpu

from tests.gpu_util import GpuRun, assert_close  # noqa: E402


def test_cfg1_full():
    e, args, df = W.workload("cfg1", full=True)
    run = GpuRun(e, args, df)
    orc = Oracle(e)
    f_o, fabs = orc.forward(args)
    assert_close(run.forward(), f_o, fabs, "cfg1 forward")
    dx_o, t_o = orc.backward(args, df)
    for g, o, t, n in zip(run.backward(), dx_o, t_o, e.arg_names):
        assert_close(g, o, t, f"cfg1 d{n}")


def test_cfg2_full_sampled():
    e, args, df = W.workload("cfg2", full=True)
    run = GpuRun(e, args, df)
    f_g = run.forward()
    da, db, dc, dd = run.backward()
    orc = Oracle(e)
    nt = max_threads()
    ni, nj, nk = 8192, 8192, 32
    # rows i in [i0, i1): a[i;k], c[i;i] are read only by alpha with that i; d[i+k] by i in [beta-31, beta]
    for i0, i1 in [(0, 40), (4093, 4133), (8152, 8192)]:
        lo, hi = [i0, 0], [i1, nj]
        f_o, fabs = orc.forward(args, lo, hi, nthreads=nt)
        assert_close(f_g[i0:i1], f_o[i0:i1], fabs[i0:i1], "cfg2 forward rows")
        dx_o, t_o = orc.backward(args, df, lo, hi, wanted=[True, False, True, True], nthreads=nt)
        assert_close(da[i0:i1], dx_o[0][i0:i1], t_o[0][i0:i1], "cfg2 da rows")
        diag = np.arange(i0, i1)
        assert_close(dc[diag, diag], dx_o[2][diag, diag], t_o[2][diag, diag], "cfg2 dc diagonal")
        b0 = 0 if i0 == 0 else i0 + nk - 1          # every i that reaches beta lies in the sub-box
        b1 = ni + nk - 2 if i1 == ni else i1 - 1
        assert_close(dd[b0:b1 + 1], dx_o[3][b0:b1 + 1], t_o[3][b0:b1 + 1], "cfg2 dd")
    # columns j in [j0, j1): b[j;k] is read only by alpha with that j
    for j0, j1 in [(0, 24), (8168, 8192)]:
        dx_o, t_o = orc.backward(args, df, [0, j0], [ni, j1], wanted=[False, True, False, False], nthreads=nt)
        assert_close(db[j0:j1], dx_o[1][j0:j1], t_o[1][j0:j1], "cfg2 db rows")
    # off-diagonal elements of dc have an empty Gamma: exactly zero everywhere
    assert np.count_nonzero(dc) <= ni
    off = dc.copy()
    off[np.arange(ni), np.arange(ni)] = 0
    assert not off.any()
    assert np.isfinite(f_g).all() and np.isfinite(da).all() and np.isfinite(db).all() and np.isfinite(dd).all()


def test_cfg3_full():
    e, args, df = W.workload("cfg3", full=True)
    run = GpuRun(e, args, df)
    orc = Oracle(e)
    nt = max_threads()
    f_o, fabs = orc.forward(args, nthreads=nt)
    assert_close(run.forward(), f_o, fabs, "cfg3 forward")
    dx_o, t_o = orc.backward(args, df, nthreads=nt)
    dx, dW = run.backward()
    assert_close(dx, dx_o[0], t_o[0], "cfg3 dx")
    assert_close(dW, dx_o[1], t_o[1], "cfg3 dW")
    assert dx[20476] == 0.0 and dx[20477] == 0.0       # never read
    assert np.count_nonzero(dW) <= 4096


def test_cfg4_full():
    e, args, df = W.workload("cfg4", full=True)
    run = GpuRun(e, args, df)
    orc = Oracle(e)
    nt = max_threads()
    f_g = run.forward()
    dx, dy = run.backward()
    f_o, fabs = orc.forward(args, nthreads=nt)
    assert_close(f_g, f_o, fabs, "cfg4 forward")
    del f_o, fabs, f_g
    dx_o, t_o = orc.backward(args, df, nthreads=nt)
    assert_close(dx, dx_o[0], t_o[0], "cfg4 dx")
    assert_close(dy, dx_o[1], t_o[1], "cfg4 dy")
    assert not dy[np.arange(1534) % 3 != 0].any()      # 3 does not divide beta: masked
    assert not dx[1534].any()                          # the last row of x is never read


def test_cfg5_full_sampled():
    e, args, df = W.workload("cfg5", full=True)
    run = GpuRun(e, args, df)
    f_g = run.forward()
    dx, dw = run.backward()
    orc = Oracle(e)
    nt = max_threads()
    nb, no, ntime = 64, 256, 2048
    # batch b0: x[b0] is read only by alpha with b = b0, so dx[b0] is complete in this sub-box
    for b0 in (0, 37):
        lo, hi = [b0, 0, 0], [b0 + 1, no, ntime]
        f_o, fabs = orc.forward(args, lo, hi, nthreads=nt)
        assert_close(f_g[b0], f_o[b0], fabs[b0], "cfg5 forward batch")
        dx_o, t_o = orc.backward(args, df, lo, hi, wanted=[True, False], nthreads=nt)
        assert_close(dx[b0], dx_o[0][b0], t_o[0][b0], "cfg5 dx batch")
    # output channel o0: w[o0] is read only by alpha with o = o0
    for o0 in (0, 255):
        dx_o, t_o = orc.backward(args, df, [0, o0, 0], [nb, o0 + 1, ntime], wanted=[False, True], nthreads=nt)
        assert_close(dw[o0], dx_o[1][o0], t_o[1][o0], "cfg5 dw channel")
    assert np.isfinite(dx).all() and np.isfinite(dw).all() and np.isfinite(f_g).all()
    # bilinearity: <df, f(x, w)> = <dx, x> = <dw, w>  (float64 accumulation of fp32 results)
    lhs = float(np.dot(df.numpy().reshape(-1).astype(np.float64), f_g.reshape(-1).astype(np.float64)))
    r1 = float(np.dot(dx.reshape(-1).astype(np.float64), args[0].numpy().reshape(-1).astype(np.float64)))
    r2 = float(np.dot(dw.reshape(-1).astype(np.float64), args[1].numpy().reshape(-1).astype(np.float64)))
    scale = float(np.abs(df.numpy()).astype(np.float64).sum()) * 1e-5
    assert abs(lhs - r1) <= scale and abs(lhs - r2) <= scale

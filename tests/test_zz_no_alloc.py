"""tad_backward_noalloc: the gradient entry point for callers that cannot allocate device memory
(it keeps its scratch in a fixed array inside the library).  Its results must equal those of
tad_backward with a caller-provided workspace, also when it is called twice in a row, because
the second call finds the first call's leftovers in the shared array.  Collected last on
purpose, so that a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from workloads import configs as W

pytestmark = pytest.mark.gpu

from paper_1711_01348_b200 import Plan, TadError  # noqa: E402
from tests.gpu_util import GpuRun, assert_close  # noqa: E402
from oracle.oracle import Oracle  # noqa: E402


def _noalloc(run):
    stream = torch.cuda.current_stream().cuda_stream
    out = [torch.full_like(d, float("nan")) for d in run.dargs]
    run.plan.backward_noalloc([a.data_ptr() for a in run.args], run.df.data_ptr(),
                              [o.data_ptr() for o in out], stream)
    torch.cuda.synchronize()
    return [o.cpu().numpy() for o in out]


@pytest.mark.parametrize("debug_bounds", [False, True])
def test_noalloc_matches_workspace_entry_point_twice(debug_bounds):
    e, args, df = W.workload("cfg2", full=False)          # its gradients read a staged adjoint
    run = GpuRun(e, args, df, debug_bounds=debug_bounds)
    assert run.plan.num_stages() == 1 and run.plan.workspace_bytes() > 0
    want = run.backward()
    _, t_o = Oracle(e).backward(args, df)
    for call in range(2):
        got = _noalloc(run)
        # the debug word of this entry point lives in its own scratch: a NULL workspace asks about that one
        run.plan.debug_status(0)
        for g, w, t, name in zip(got, want, t_o, e.arg_names):
            assert_close(g, w.astype(np.float64), t, f"noalloc call {call} d{name}")
            np.testing.assert_array_equal(g, w)            # same kernels, same order: bitwise equal
    # a different plan afterwards sees the previous plan's contents in the shared array
    e2, args2, df2 = W.workload("cfg1", full=True)
    run2 = GpuRun(e2, args2, df2)
    want2 = run2.backward()
    for g, w in zip(_noalloc(run2), want2):
        np.testing.assert_array_equal(g, w)


def test_noalloc_rejects_plans_beyond_its_scratch():
    e = W.FULL["cfg2"]()                                   # needs 256 MiB of scratch
    plan = Plan(e)
    assert plan.workspace_bytes() > 32 * 1024 * 1024
    with pytest.raises(TadError) as ei:
        plan.backward_noalloc([0] * 4, 0, [0] * 4)
    assert ei.value.code == "TAD_ERR_WORKSPACE" and "at most" in str(ei.value)

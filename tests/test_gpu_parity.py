"""Parity of the CUDA path with the float64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle.oracle import Oracle, max_threads
from workloads import configs as W

pytestmark = pytest.mark.gpu

from tests.gpu_util import GpuRun, assert_close, check_against_oracle  # noqa: E402

SMALL = {
    "sec6": (lambda: W.ex_section6(), ("uniform", -0.5, 0.5)),
    "square_broadcast": (lambda: W.ex_square_broadcast(70, 133), ("uniform", -1, 1)),
    "diag_square": (lambda: W.ex_diag_square(77), ("uniform", -1, 1)),
    "exp_shift": (lambda: W.ex_exp_shift(150, 67), ("uniform", -1, 1)),
    "sin": (lambda: W.ex_sin(1000), ("normal", 0, 1)),
    "xy": (lambda: W.ex_xy(131), ("normal", 0, 1)),
    "diag_cube": (lambda: W.ex_diag_cube(45), ("normal", 0, 1)),
    "matmul": (lambda: W.ex_matmul(37, 150, 41), ("normal", 0, 1)),
    "exp_flat": (lambda: W.ex_exp_flat(33, 7), ("uniform", -1, 1)),
    "strided": (lambda: W.ex_strided(301, 2), ("normal", 0, 1)),
    "strided3": (lambda: W.ex_strided(100, 3), ("normal", 0, 1)),
    "strided2": (lambda: W.ex_strided2(40, 33), ("normal", 0, 1)),
    "lattice2d": (lambda: W.ex_lattice2d(35, 44), ("normal", 0, 1)),
    "all_ops": (lambda: W.ex_all_ops(300), ("uniform", -0.9, 0.9)),
    "tiny": (lambda: W.intro(1, 1, 1), ("uniform", -0.5, 0.5)),
    "one_row": (lambda: W.intro(1, 200, 3), ("uniform", -0.5, 0.5)),
    "one_col": (lambda: W.intro(200, 1, 3), ("uniform", -0.5, 0.5)),
}


@pytest.mark.parametrize("name", sorted(SMALL))
def test_small_expressions(name):
    make, dist = SMALL[name]
    e = make()
    args, df = W.make_inputs(e, dist, seed=0)
    check_against_oracle(e, args, df, debug_bounds=True)
    check_against_oracle(e, args, df)


# Sizes at which the compiler picks its wide vector shapes (4x8, 2x8, 1x8, 1x4, 16x1 values per thread),
# split summations and fused inner loops, with extents that leave a ragged tail in every direction.
MID = {
    "intro_mid": (lambda: W.intro(300, 333, 11), ("uniform", -0.5, 0.5)),
    "intro_wide": (lambda: W.intro(130, 1000, 21), ("uniform", -0.5, 0.5)),
    "matmul_t": (lambda: W.ex_matmul_t(70, 100, 37), ("normal", 0, 1)),
    "rowsum_sq": (lambda: W.ex_rowsum_sq(1000, 37), ("normal", 0, 1)),
    "rowsum_sq_short": (lambda: W.ex_rowsum_sq(333, 9), ("normal", 0, 1)),
    "conv_mid": (lambda: W.conv1d(3, 20, 24, 300, 5), ("normal", 0, 0.1)),
    "matmul_mid": (lambda: W.ex_matmul(150, 67, 1100), ("normal", 0, 1)),
    # large enough for the 4 x 8 product shape: forward and dw (outer product and per-element operand,
    # ragged tails along t), then dw and dx with the lanes along c and per-u tap ranges (masked trips)
    "conv_wide": (lambda: W.conv1d(16, 4, 128, 2400, 5), ("normal", 0, 0.1)),
    "conv_channels": (lambda: W.conv1d(4, 160, 24, 700, 3), ("normal", 0, 0.1)),
    # four gradient elements per thread of which the first has no term, and a function of a sum
    # that is evaluated once for the four
    "guarded_shared_fn": (lambda: W.ex_guarded_shared_fn(55, 160, 5, 15), ("uniform", -1, 1)),
}


@pytest.mark.parametrize("name", sorted(MID))
def test_mid_size_expressions(name):
    make, dist = MID[name]
    e = make()
    args, df = W.make_inputs(e, dist, seed=1)
    check_against_oracle(e, args, df, nthreads=max_threads())


@pytest.mark.parametrize("key", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_reduced_workloads(key):
    """Same structure as the full workloads, several tiles and ragged tails, full oracle run."""
    e, args, df = W.workload(key, full=False)
    check_against_oracle(e, args, df, nthreads=max_threads(), debug_bounds=True)
    check_against_oracle(e, args, df, nthreads=max_threads())


@pytest.mark.parametrize("fn", ["exp", "log", "sin", "cos", "tanh", "sinh", "cosh"])
def test_function_argument_sweeps(fn):
    """The inline evaluations (own range reduction, polynomials, fast exponential) and the library
    fall-backs, over large, tiny and awkward arguments, value and derivative."""
    e, args, df = W.function_sweep(fn)
    check_against_oracle(e, args, df)


@pytest.mark.parametrize("name", ["sec6", "exp_shift", "exp_flat", "all_ops", "one_row"])
def test_saved_forward_small(name):
    """Plans that read the forward output instead of evaluating the expression again in the derivative."""
    make, dist = SMALL[name]
    e = make()
    args, df = W.make_inputs(e, dist, seed=2)
    check_against_oracle(e, args, df, saved_forward=True)
    check_against_oracle(e, args, df, saved_forward=True, debug_bounds=True)


@pytest.mark.parametrize("key", ["cfg1", "cfg2", "cfg3", "cfg5"])
def test_saved_forward_reduced_workloads(key):
    e, args, df = W.workload(key, full=False)
    check_against_oracle(e, args, df, nthreads=max_threads(), saved_forward=True)


def test_saved_forward_needs_f():
    from paper_1711_01348_b200 import TadError
    e, args, df = W.workload("cfg1", full=False)
    run = GpuRun(e, args, df, saved_forward=True)
    with pytest.raises(TadError):
        run.plan.backward([a.data_ptr() for a in run.args] + [0], run.df.data_ptr(), [d.data_ptr() for d in run.dargs],
                          run.ws.data_ptr(), run.ws.numel())


def test_gradient_subset_and_repeat_calls():
    e, args, df = W.workload("cfg2", full=False)
    run = GpuRun(e, args, df)
    first = run.backward()
    only_b = run.backward(wanted=[False, True, False, False])
    np.testing.assert_array_equal(first[1], only_b[1])
    second = run.backward()
    for a, b in zip(first, second):
        np.testing.assert_array_equal(a, b)       # fixed summation order: bitwise repeatable


def test_null_pointer_is_rejected():
    from paper_1711_01348_b200 import TadError
    e, args, df = W.workload("cfg1", full=False)
    run = GpuRun(e, args, df)
    with pytest.raises(TadError):
        run.plan.forward([a.data_ptr() for a in run.args], 0)
    with pytest.raises(TadError):
        run.plan.backward([0] * 4, run.df.data_ptr(), [d.data_ptr() for d in run.dargs])


@pytest.mark.parametrize("key,saved", [("cfg2", False), ("cfg2", True), ("cfg4", False), ("cfg5", False)])
def test_host_buffer_entry_point(key, saved):
    """tad_step_host: host buffers in, forward and every gradient back, copies inside the call."""
    from paper_1711_01348_b200 import Plan
    e, args, df = W.workload(key, full=False)
    plan = Plan(e, saved_forward=saved)
    h_args = [a.contiguous().pin_memory() for a in args]
    h_df = df.contiguous().pin_memory()
    h_f = torch.full(list(e.out_shape), float("nan"), dtype=torch.float32).pin_memory()
    h_dargs = [torch.full(list(s), float("nan"), dtype=torch.float32).pin_memory() for s in e.arg_shapes]
    staging = torch.empty(plan.staging_bytes(), dtype=torch.uint8, device="cuda:0")
    for _ in range(2):           # the staging area is reused as it stands
        plan.step_host([a.data_ptr() for a in h_args], h_df.data_ptr(), h_f.data_ptr(),
                       [d.data_ptr() for d in h_dargs], staging.data_ptr(), staging.numel(),
                       torch.cuda.current_stream().cuda_stream)
    orc = Oracle(e)
    f_o, fabs_o = orc.forward(args, nthreads=max_threads())
    assert_close(h_f.numpy(), f_o, fabs_o, f"{e.name} forward (host buffers)")
    dx_o, t_o = orc.backward(args, df, nthreads=max_threads())
    for p, name in enumerate(e.arg_names):
        assert_close(h_dargs[p].numpy(), dx_o[p], t_o[p], f"{e.name} d{name} (host buffers)")


@pytest.mark.parametrize("seed", range(80))
def test_random_expressions(seed):
    """Random index maps (strides, negative and repeated indices, several index expressions of one
    argument) and random function trees, every gradient against the oracle."""
    from paper_1711_01348_b200 import TadError
    from workloads.random_expr import random_expression
    e = random_expression(seed)
    args, df = W.make_inputs(e, ("uniform", -1, 1), seed=seed)
    try:
        check_against_oracle(e, args, df, debug_bounds=seed % 3 == 0, saved_forward=seed % 4 == 1)
    except TadError as exc:
        if "TAD_ERR_UNSUPPORTED" in str(exc) or "TAD_ERR_OVERFLOW" in str(exc):
            pytest.skip(str(exc))
        raise


@pytest.mark.parametrize("seed", range(40))
def test_random_expressions_large(seed):
    """The same at extents where the wide vector shapes, element variables and split summations apply."""
    from paper_1711_01348_b200 import TadError
    from workloads.random_expr import random_expression
    e = random_expression(seed, large=1)
    args, df = W.make_inputs(e, ("uniform", -1, 1), seed=seed)
    try:
        check_against_oracle(e, args, df, nthreads=max_threads(), saved_forward=seed % 4 == 1)
    except TadError as exc:
        if "TAD_ERR_UNSUPPORTED" in str(exc) or "TAD_ERR_OVERFLOW" in str(exc):
            pytest.skip(str(exc))
        raise


@pytest.mark.parametrize("seed", range(12))
def test_random_expressions_huge(seed):
    """... and with millions of outputs: 16 values per thread, element variables, fused loops."""
    from paper_1711_01348_b200 import TadError
    from workloads.random_expr import random_expression
    e = random_expression(seed, large=2)
    args, df = W.make_inputs(e, ("uniform", -1, 1), seed=seed)
    try:
        check_against_oracle(e, args, df, nthreads=max_threads(), saved_forward=seed % 4 == 1)
    except TadError as exc:
        if "TAD_ERR_UNSUPPORTED" in str(exc) or "TAD_ERR_OVERFLOW" in str(exc):
            pytest.skip(str(exc))
        raise


def _conditioning(e, args, df, nthreads):
    """Decided by the oracle alone, element by element: with the arguments moved by eight fp32 rounding steps
    (relative 2^-20, random signs, three independent draws: what a sum of some dozens of rounded terms
    accumulates) an element is well-conditioned when its result moves by at most a quarter of the tolerance
    in every draw.  Deep compositions (a function of a long cancelling sum, 1 - tanh^2 at saturation) leave it
    on any fp32 code.  Returns the oracle's results, the masks of well-conditioned elements (f first, then the
    gradients) and the fraction of elements they cover."""
    from tests.gpu_util import ATOL, RTOL_TERMS
    orc = Oracle(e)
    f0, s0 = orc.forward(args, nthreads=nthreads)
    d0, t0 = orc.backward(args, df, nthreads=nthreads)
    # three independent draws of the signs: one draw alone leaves an element whose perturbations happen to cancel
    masks = None
    for draw in range(3):
        rng = np.random.default_rng(12345 + draw)
        moved = [a.numpy().astype(np.float64) * (1.0 + 2.0 ** -20 * rng.choice([-1.0, 1.0], size=tuple(a.shape))) for a in args]
        f1, _ = orc.forward(moved, nthreads=nthreads)
        d1, _ = orc.backward(moved, df, nthreads=nthreads)
        with np.errstate(all="ignore"):
            pairs = [(f0, f1, s0)] + [(d0[p], d1[p], t0[p]) for p in range(len(args))]
            ok = [np.abs(a - b) <= 0.25 * (RTOL_TERMS * sc + ATOL) for a, b, sc in pairs]
        masks = ok if masks is None else [m & o for m, o in zip(masks, ok)]
    covered = sum(int(m.sum()) for m in masks) / max(1, sum(m.size for m in masks))
    return (f0, s0, d0, t0), masks, covered


def _check_conditioned(e, args, df, seed):
    """Every well-conditioned element is compared; a draw in which fewer than 90 % of the elements are
    well-conditioned fails (the generator is meant to produce expressions fp32 can evaluate)."""
    from paper_1711_01348_b200 import TadError
    results, masks, covered = _conditioning(e, args, df, max_threads())
    assert covered >= 0.9, f"only {covered:.1%} of the elements are well-conditioned in fp32"
    try:
        check_against_oracle(e, args, df, nthreads=max_threads(), saved_forward=seed % 4 == 1,
                             oracle_results=results, masks=masks)
    except TadError as exc:
        if "TAD_ERR_UNSUPPORTED" in str(exc) or "TAD_ERR_OVERFLOW" in str(exc):
            pytest.skip(str(exc))
        raise


@pytest.mark.parametrize("seed", range(120))
def test_random_expressions_nested_sums(seed):
    """A sum of up to 40 terms inside a sum of up to 12, index expressions at every depth (some of
    them independent of the sums that enclose them)."""
    from workloads.random_expr import random_expression
    e = random_expression(seed, large=3)
    args, df = W.make_inputs(e, ("uniform", -1, 1), seed=seed)
    _check_conditioned(e, args, df, seed)


@pytest.mark.parametrize("seed", range(50))
def test_random_expressions_all_functions(seed):
    """One or two sums (the inner one up to 64 terms), up to 2e5 outputs, and log, division, sinh and
    cosh among the functions, their arguments kept inside their domains."""
    from workloads.random_expr import random_expression
    e = random_expression(seed, large=4)
    args, df = W.make_inputs(e, ("uniform", -1, 1), seed=seed)
    _check_conditioned(e, args, df, seed)


@pytest.mark.parametrize("seed", range(40))
def test_random_contractions(seed):
    """Products of two index expressions under one or two sums, 4e4 to 4e6 outputs: the product
    kernels (32 sums per thread) and the shapes next to them, with random strides and offsets."""
    from workloads.random_expr import random_expression
    e = random_expression(seed, large=5)
    args, df = W.make_inputs(e, ("normal", 0, 1), seed=seed)
    check_against_oracle(e, args, df, nthreads=max_threads(), saved_forward=seed % 4 == 1)


@pytest.mark.parametrize("level,seed", [(lv, sd) for lv in (0, 1, 3, 4) for sd in range(12)])
def test_entry_points_agree(level, seed):
    """tad_backward with every gradient, with a subset of them (the others untouched), the entry point
    with its own scratch and the host-buffer step run the same kernels: bit-identical results."""
    from paper_1711_01348_b200 import TadError
    from workloads.random_expr import random_expression
    e = random_expression(seed, large=level)
    args, df = W.make_inputs(e, ("normal", 0, 0.7), seed=seed)
    saved = seed % 2 == 1
    try:
        run = GpuRun(e, args, df, saved_forward=saved)
    except TadError as exc:
        if "TAD_ERR_UNSUPPORTED" in str(exc) or "TAD_ERR_OVERFLOW" in str(exc):
            pytest.skip(str(exc))
        raise
    f = run.forward()
    d = run.backward()
    stream = torch.cuda.current_stream().cuda_stream
    extra = [run.f.data_ptr()] if saved else []
    if run.plan.workspace_bytes() <= 32 << 20:
        outs = [torch.full(list(s), float("nan"), dtype=torch.float32, device="cuda:0") for s in e.arg_shapes]
        run.plan.backward_noalloc([x.data_ptr() for x in run.args] + extra, run.df.data_ptr(),
                                  [o.data_ptr() for o in outs], stream)
        torch.cuda.synchronize()
        for p, o in enumerate(outs):
            assert np.array_equal(o.cpu().numpy(), d[p], equal_nan=True), f"own scratch, gradient {p}"
    wanted = [(seed >> p) & 1 == 0 for p in range(len(e.arg_shapes))]
    other = GpuRun(e, args, df, saved_forward=saved)
    other.forward()
    sub = other.backward(wanted)
    for p, w in enumerate(wanted):
        if w:
            assert np.array_equal(sub[p], d[p], equal_nan=True), f"subset, gradient {p}"
        else:
            assert np.all(np.isnan(other.dargs[p].cpu().numpy())), f"gradient {p} was not asked for but written"
    h_args = [x.contiguous().pin_memory() for x in args]
    h_df = df.contiguous().pin_memory()
    h_f = torch.full(list(e.out_shape), float("nan"), dtype=torch.float32).pin_memory()
    h_d = [torch.full(list(s), float("nan"), dtype=torch.float32).pin_memory() for s in e.arg_shapes]
    staging = torch.empty(run.plan.staging_bytes(), dtype=torch.uint8, device="cuda:0")
    run.plan.step_host([x.data_ptr() for x in h_args], h_df.data_ptr(), h_f.data_ptr(), [x.data_ptr() for x in h_d],
                       staging.data_ptr(), staging.numel(), stream)
    assert np.array_equal(h_f.numpy(), f, equal_nan=True), "host buffers, f"
    for p in range(len(h_d)):
        assert np.array_equal(h_d[p].numpy(), d[p], equal_nan=True), f"host buffers, gradient {p}"

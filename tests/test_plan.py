"""Compiled plans against brute force: for every index expression and every argument element the
set Gamma-hat(beta) that the plan enumerates (mask, index transform, bound rows) must equal the
set of alpha_hat that map to beta, bit-exactly.  Host only."""
import itertools
import os

import numpy as np
import pytest

from oracle.oracle import Oracle
from paper_1711_01348_b200 import EXPORTS, Plan, TadError, lib
from workloads import configs as W
from workloads.expr import Builder, unit


def brute_force_gamma(e, q):
    """dict beta -> sorted list of alpha_hat (restricted to output indices + enclosing sums)."""
    acc = e.accesses[q]
    n_out = len(e.out_shape)
    # enclosing sums of the loads that use this index expression
    encl = set()

    def walk(n, stack):
        nd = e.nodes[n]
        if nd.op == "load":
            if nd.access == q:
                encl.update(stack)
            return
        if nd.op == "sum":
            walk(nd.in0, stack + [n])
            return
        for c in (nd.in0, nd.in1):
            if c >= 0:
                walk(c, stack)
    walk(len(e.nodes) - 1, [])
    sums = sorted(encl, key=lambda n: e.nodes[n].sum_idx)
    pos = list(range(n_out)) + [e.nodes[n].sum_idx for n in sums]
    ranges = [range(s) for s in e.out_shape] + [range(e.nodes[n].sum_lo, e.nodes[n].sum_hi + 1) for n in sums]
    out = {}
    A = np.array(acc.A)[:, pos]
    off = np.array(acc.offset)
    for ah in itertools.product(*ranges):
        beta = tuple(int(v) for v in A.dot(np.array(ah)) + off)
        out.setdefault(beta, []).append(tuple(ah))
    return pos, out


SMALL = {
    "sec6": lambda: W.ex_section6(),
    "intro": lambda: W.intro(5, 4, 3),
    "shifted": lambda: W.shifted(7),
    "nonunimodular": lambda: W.nonunimodular(4),
    "conv1d": lambda: W.conv1d(2, 3, 2, 6, 5),
    "square_broadcast": lambda: W.ex_square_broadcast(4, 5),
    "diag_square": lambda: W.ex_diag_square(5),
    "exp_shift": lambda: W.ex_exp_shift(4, 6),
    "matmul": lambda: W.ex_matmul(3, 4, 5),
    "exp_flat": lambda: W.ex_exp_flat(4, 3),
    "strided": lambda: W.ex_strided(5, 2),
    "strided2": lambda: W.ex_strided2(4, 3),
    "lattice2d": lambda: W.ex_lattice2d(4, 3),
    "all_ops": lambda: W.ex_all_ops(4),
}


@pytest.mark.parametrize("name", sorted(SMALL))
def test_gamma_sets_match_brute_force(name):
    e = SMALL[name]()
    plan = Plan(e)
    orc = Oracle(e)
    for q, acc in enumerate(e.accesses):
        pos, want = brute_force_gamma(e, q)
        info = plan.access_info(q)
        assert list(info.idx_pos)[:info.n_idx] == pos
        counts = orc.counts(q)
        shape = e.arg_shapes[acc.arg]
        for beta in itertools.product(*[range(s) for s in shape]):
            n, got = plan.enumerate(q, beta, cap=4096)
            exp = sorted(want.get(beta, []))
            assert n == len(exp) == int(counts[beta]), (name, q, beta)
            assert sorted(got) == exp, (name, q, beta)


def _mat(buf, r, c):
    return np.array([[buf[i * c + j] for j in range(c)] for i in range(r)], dtype=object)


@pytest.mark.parametrize("name", sorted(SMALL) + ["cfg2_full", "cfg3_full", "cfg4_full", "cfg5_full"])
def test_plan_invariants(name):
    e = SMALL[name]() if name in SMALL else W.FULL[name[:4]]()
    plan = Plan(e)
    for q in range(len(e.accesses)):
        i = plan.access_info(q)
        A = _mat(i.A, i.rank, i.n_idx); U = _mat(i.U, i.rank, i.rank); V = _mat(i.V, i.n_idx, i.n_idx)
        S = U.dot(A).dot(V)
        for r in range(i.rank):
            for c in range(i.n_idx):
                assert S[r, c] == (i.S[r] if (r == c and r < i.R) else 0)
        assert all(i.S[r] > 0 for r in range(i.R))
        assert all(i.S[r + 1] % i.S[r] == 0 for r in range(i.R - 1))
        assert abs(round(np.linalg.det(np.array(V, dtype=np.float64)))) == 1
        assert abs(round(np.linalg.det(np.array(U, dtype=np.float64)))) == 1
        assert i.kappa == i.n_idx - i.R
        assert bool(i.masked) == (i.R < i.rank or any(i.S[r] != 1 for r in range(i.R)))
        for l in range(i.kappa):
            assert i.n_lower[l] >= 1 and i.n_upper[l] >= 1


def test_section6_printed_ranges(golden_dir):
    """Sizes of the printed summation ranges (the kernel basis is not unique, the counts are)."""
    e = W.ex_section6()
    plan = Plan(e)
    q_of = {e.arg_names[a.arg]: q for q, a in enumerate(e.accesses)}
    golden = None
    for line in open(os.path.join(golden_dir, "section6_ranges.txt")):
        tok = line.split()
        if tok[:2] == ["dd", "counts"]:
            golden = [int(t) for t in tok[2:]]
    assert [plan.count(q_of["d"], [b]) for b in range(8)] == golden
    # da: sum over z0 = 0..3 ; db: 0..2 ; dc: delta(dc_0 - dc_1) * (5 * 4)
    assert all(plan.count(q_of["a"], [i, k]) == 4 for i in range(3) for k in range(5))
    assert all(plan.count(q_of["b"], [j, k]) == 3 for j in range(4) for k in range(5))
    for c0 in range(3):
        for c1 in range(3):
            assert plan.count(q_of["c"], [c0, c1]) == (20 if c0 == c1 else 0)
    # dd reads df at [dd_0 - z1 ; z0]: every enumerated alpha_hat has i + k = dd_0
    for b in range(8):
        _, pts = plan.enumerate(q_of["d"], [b], cap=64)
        assert all(i + k == b and 0 <= j <= 3 for (i, j, k) in pts)
    # rank-1 map of c[i;i]: one cokernel row proportional to (1, -1)
    ic = plan.access_info(q_of["c"])
    assert ic.R == 1 and ic.rank == 2 and ic.masked == 1
    C = [ic.U[1 * 2 + 0], ic.U[1 * 2 + 1]]
    assert C[0] == -C[1] and abs(C[0]) == 1


def test_divisibility_is_kept():
    """f_i = x_{2i}: odd elements pass every range test but have no integer pre-image."""
    e = W.ex_strided(5, 2)
    plan = Plan(e)
    assert [plan.count(0, [b]) for b in range(9)] == [1, 0, 1, 0, 1, 0, 1, 0, 1]
    e = W.ex_strided2(4, 3)
    plan = Plan(e)
    info = plan.access_info(0)
    assert info.S[0] == 2 and info.masked == 1
    for b in range(e.arg_shapes[0][0]):
        if b % 2:
            assert plan.count(0, [b]) == 0


@pytest.mark.parametrize("key", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_counts_sampled(key):
    """Closed-form term counts at full size on sampled elements."""
    e = W.FULL[key]()
    plan = Plan(e)
    rng = np.random.default_rng(3)
    if key == "cfg2":
        q = {e.arg_names[a.arg]: i for i, a in enumerate(e.accesses)}
        assert plan.count(q["a"], [17, 5]) == 8192 and plan.count(q["b"], [8191, 31]) == 8192
        assert plan.count(q["c"], [100, 100]) == 8192 * 32 and plan.count(q["c"], [100, 101]) == 0
        for b in [0, 1, 30, 31, 32, 4000, 8191, 8192, 8221, 8222]:
            ks = min(31, b) - max(0, b - 8191) + 1
            assert plan.count(q["d"], [b]) == max(0, ks) * 8192
    if key == "cfg3":
        n = 4096
        for b in [int(v) for v in rng.integers(0, 20478, 40)] + [0, 8190, 20475, 20476, 20477]:
            c0 = max(0, min(b, n - 1) - max(0, b - n + 1) + 1)
            assert plan.count(0, [b]) == c0
            c1 = sum(1 for j in range(n) if b - 3 * j >= 0 and (b - 3 * j) % 2 == 0 and (b - 3 * j) // 2 < n)
            assert plan.count(1, [b]) == c1
        assert plan.count(2, [7, 7]) == n and plan.count(2, [7, 8]) == 0
    if key == "cfg4":
        n = 512
        for _ in range(40):
            b0, b1 = int(rng.integers(0, 3 * n - 1)), int(rng.integers(0, 2 * n - 1))
            c = sum(1 for i in range(n) if 0 <= b0 - 2 * i < n and 0 <= (b0 - 2 * i) - b1 + n - 1 < n)
            assert plan.count(0, [b0, b1]) == c
        assert plan.count(1, [3 * 77]) == n * n and plan.count(1, [3 * 77 + 1]) == 0
    if key == "cfg5":
        # x[b; c; p]: 256 output channels times the taps u with p - u even and t in range
        qx = [i for i, a in enumerate(e.accesses) if e.arg_names[a.arg] == "x"][0]
        qw = [i for i, a in enumerate(e.accesses) if e.arg_names[a.arg] == "w"][0]
        for p_ in [0, 1, 2, 3, 4, 5, 2000, 4093, 4094, 4095, 4096, 4097, 4098]:
            c = sum(1 for u in range(5) if (p_ - u) >= 0 and (p_ - u) % 2 == 0 and (p_ - u) // 2 < 2048)
            assert plan.count(qx, [3, 200, p_]) == 256 * c
        assert plan.count(qw, [5, 6, 4]) == 64 * 2048


def test_compile_errors():
    # read outside the argument
    e = W.ex_exp_shift(4, 4)
    e.arg_shapes[0] = [5]
    with pytest.raises(TadError) as ei:
        Plan(e)
    assert ei.value.code == "TAD_ERR_OUT_OF_RANGE"
    # operand that is not an earlier node
    e = W.ex_sin(4)
    e.nodes[1].in0 = 1
    with pytest.raises(TadError) as ei:
        Plan(e)
    assert ei.value.code == "TAD_ERR_BAD_EXPR"
    # sum index used outside its sum
    b = Builder("bad", [4], 1, ["x"], [[8]])
    ld = b.load("x", [unit(2, (0, 1), (1, 1))])
    s = b.sum(1, 0, 3, b.const(1.0))
    b.bin("add", ld, s)
    with pytest.raises(TadError) as ei:
        Plan(b.done())
    assert ei.value.code == "TAD_ERR_BAD_EXPR"
    # tensor with 2^31 elements
    e = W.ex_sin(4)
    e.arg_shapes[0] = [1 << 31]
    with pytest.raises(TadError) as ei:
        Plan(e)
    assert ei.value.code == "TAD_ERR_OVERFLOW"
    # node shared between two different sets of enclosing sums
    b = Builder("shared", [4], 1, ["x"], [[4]])
    ld = b.load("x", [unit(2, (0, 1))])
    s = b.sum(1, 0, 3, ld)
    b.bin("add", ld, s)
    with pytest.raises(TadError) as ei:
        Plan(b.done())
    assert ei.value.code == "TAD_ERR_UNSUPPORTED"


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(os.path.dirname(__file__), "..", "include", "tad.h")).read()
    import re
    declared = set(re.findall(r"\b(tad_[a-z_0-9]+)\s*\(", header))
    declared -= {"tad_status"}
    assert declared == set(EXPORTS), declared ^ set(EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_kernel_stats_and_listing():
    e = W.FULL["cfg2"]()
    plan = Plan(e)
    fwd = plan.kernel_stats(-1)
    # the sum over k is pushed inside the term and the kernel is one contraction with exp(-.) as its epilogue: 32
    # summation indices for a_ik b_jk plus one each for the terms that depend on i only and on i and j separately;
    # before it, small kernels pre-evaluate those terms and the two operand matrices
    assert fwd.outputs == 8192 * 8192 and fwd.n_launches == 7
    listing = plan.disassemble(-1)
    assert "; factored" in listing and "; contraction 8192 x 8192 x 34" in listing and "2 epilogue steps" in listing
    # forward: per (i,j,k) add, square, multiply, add, accumulate (5) + cube per (i,k) + neg, exp per (i,j)
    nij, nk = 8192.0 * 8192.0, 32.0
    assert fwd.alg_flops == pytest.approx(5 * nij * nk + 2 * 8192 * nk + 2 * nij, rel=1e-6)
    assert fwd.alg_bytes == pytest.approx(4 * nij + 4 * (2 * 8192 * 32 + 8223) + 32 * 8192, rel=1e-6)
    q = {e.arg_names[a.arg]: i for i, a in enumerate(e.accesses)}
    st = plan.kernel_stats(q["c"])
    # the statistics count the expression as written (no algebraic rewriting); the launches are those of the
    # factored gradient: its contractions stream the staged adjoint once (three column blocks of one matrix)
    assert st.terms == 8192 * 8192 * 32 and st.n_launches >= 4
    dc = plan.disassemble(q["c"])
    # one 32-column contraction with b, and the two single columns (plain row sums and row sums weighted by
    # sum_k b_jk^2) as passes of their own at memory speed
    assert dc.count("; contraction") == 3 and "8192 x 32 x 8192" in dc and dc.count("row sums") == 2
    # dd: the sum over j of the staged adjoint is a row sum, indexed by the row and not by (beta, z)
    dd = plan.disassemble(q["d"])
    assert "; contraction 8192 x 1 x 8192" in dd and "; line sums: 1 loads x 1 loops" in dd


# --------------------------------------------------------------------------- #
# schedules the compiler is expected to find for the workloads (read from the listings)
# --------------------------------------------------------------------------- #

def _header(listing: str) -> dict:
    # the header of the kernel itself: the last one (auxiliary kernels of the optimisation pass come first)
    first = [line for line in listing.splitlines() if line.startswith("; vars=")][-1]
    return dict(item.split("=") for item in first.lstrip("; ").split())


def test_contractions_run_on_the_tile_kernel():
    """Convolution forward and both gradients are products of two index expressions under sums: each becomes
    a contraction program.  The gradient of x has a summation whose bounds move with the gradient index as a
    band (slope 1/2): one program per residue class, three taps for even positions and two for odd ones."""
    from workloads import configs as W
    plan = Plan(W.FULL["cfg5"]())
    fwd, dw, dx = plan.disassemble(-1), plan.disassemble(0), plan.disassemble(1)
    assert fwd.count("; contraction") == 1 and "256 x 131072 x 1280" in fwd
    assert dw.count("; contraction") == 1 and "256 x 1280 x 131072" in dw and "ksplit 1 " not in dw
    assert dx.count("; contraction") == 2
    assert "x 768 " in dx and "x 512 " in dx          # 256 channels x 3 taps, x 2 taps
    assert dx.count("guard 1") == 2


def test_gradients_of_cfg3_and_cfg4_are_line_sums():
    """With exp, tanh, sin and cos tabulated over the elements of x, every gradient term of the shifted and the
    non-unimodular workload is a product of index expressions under one or two summation loops: line-sum
    programs.  Few outputs with long summations are cut into shares of about 64 terms (pieces of the loops' boxes)."""
    from workloads import configs as W
    p3 = Plan(W.FULL["cfg3"]())
    for q in (0, 1):                                  # dx through x[i + j] and through x[2i + 3j]
        text = p3.disassemble(q)
        assert "; function table" in text and "; line sums: 3 loads x 1 loops" in text and "a thread per output" in text
        assert " 1 guards" in text                    # x has elements beyond the image of i + j
    dW = p3.disassemble(2)
    assert "; line sums: 3 loads x 1 loops" in dW and "a warp per output" in dW     # df rows are read along j
    p4 = Plan(W.FULL["cfg4"]())
    dx, dy = p4.disassemble(0), p4.disassemble(1)
    assert "; line sums" in dx and " 1 shares" in dx and " 3 guards" in dx
    assert "; line sums: 2 loads x 2 loops" in dy and " 4096 shares" in dy              # 512 live outputs x 262 144 terms: 512 x 8 pieces
    assert " 64 shares" in p3.disassemble(0)                                             # ranges of up to 4 096 terms


def test_split_summations_fill_whole_waves():
    """Shares of a split summation on the interpreter: work items x shares is close to a multiple of the
    resident warps (a gradient whose term is not a plain product: the sum of two index expressions, squared)."""
    b = Builder("sq_of_sum", [2000, 2500], 0, ["x", "y"], [[2000], [4499]])
    xi = b.load("x", [unit(2, (0, 1))])
    yij = b.load("y", [unit(2, (0, 1), (1, 1))])
    b.un("exp", b.bin("add", xi, yij))
    plan = Plan(b.done())
    text = plan.disassemble(0)                     # dx_i = sum_j df_ij exp(x_i + y_{i+j}): 2000 outputs x 2500 terms
    if "; vars=" not in text:
        pytest.skip("this gradient no longer runs on the interpreter")
    head = _header(text)
    assert int(head["zsplit"]) > 1


def _lane_loop_row_variables(listing: str) -> set:
    """Variables with a non-zero coefficient in a bound row of the loop over the lane variable."""
    import re
    rows = {}
    for line in listing.splitlines():
        m = re.match(r"; row (\d+) \((-?\d+) \+ ([-\d ]+)\) / (-?\d+)", line)
        if m:
            rows[int(m.group(1))] = [int(x) for x in m.group(3).split()]
    used = set()
    for line in listing.splitlines():
        m = re.match(r"; loop \d+ var=\d+ lane=1 .* lower=(\d+)\+(\d+) upper=(\d+)\+(\d+)", line)
        if not m:
            continue
        l0, nl, u0, nu = map(int, m.groups())
        for r in list(range(l0, l0 + nl)) + list(range(u0, u0 + nu)):
            used |= {v for v, c in enumerate(rows[r]) if c}
    return used


def test_lane_loop_bounds_do_not_depend_on_the_element_variable():
    """The loop over the lane variable takes one range per thread, so a variable in its bound rows
    may not be the element variable (the thread's values would need a range each).  Seed 8 of the
    largest generator level has a gradient whose summation ranges depend on the gradient index."""
    from workloads.random_expr import random_expression
    cases = [(8, 2)] + [(s, 1) for s in range(12)] + [(s, 2) for s in range(12)]
    for seed, level in cases:
        try:
            plan = Plan(random_expression(seed, level))
        except TadError:
            continue
        for which in range(len(plan.expr.accesses)):
            listing = plan.disassemble(which)
            if "; vars=" not in listing:
                continue                              # a contraction or an element-wise program: no lane loop
            u = int(_header(listing)["unroll_var"])
            if u >= 0:
                assert u not in _lane_loop_row_variables(listing), (seed, level, which)


def test_forward_of_cfg4_is_a_table_and_an_elementwise_program():
    """The forward pass has no loops: sin over the elements of x once (a function table), then an element-wise program."""
    from workloads import configs as W
    fwd = Plan(W.FULL["cfg4"]()).disassemble(-1)
    assert "; function table" in fwd and fwd.count("; element-wise program") == 2


# --------------------------------------------------------------------------- #
# argument checks that return before anything is launched (no GPU needed)
# --------------------------------------------------------------------------- #

def _many_args(n_args):
    """f_i = x0_i + x1_i + ... : one index expression per argument."""
    from workloads.expr import Builder, unit
    b = Builder(f"sum_of_{n_args}", [8], 0, [f"x{k}" for k in range(n_args)], [[8]] * n_args)
    acc = b.load("x0", [unit(1, (0, 1))])
    for k in range(1, n_args):
        acc = b.bin("add", acc, b.load(f"x{k}", [unit(1, (0, 1))]))
    return b.done()


def test_pointer_slots_count_the_saved_forward_output():
    """Arguments, df and (for saved_forward plans) f share 16 pointer slots: 15 arguments fit without the saved
    output and are refused with it, instead of letting f overwrite the slot of df."""
    Plan(_many_args(15))
    Plan(_many_args(14), saved_forward=True)
    with pytest.raises(TadError) as ei:
        Plan(_many_args(15), saved_forward=True)
    assert ei.value.code == "TAD_ERR_UNSUPPORTED"
    with pytest.raises(TadError):
        Plan(_many_args(16))


def test_workspace_too_small_or_misaligned_is_refused_before_any_launch():
    from workloads import configs as W
    e = W.REDUCED["cfg2"]()
    plan = Plan(e)
    need = plan.workspace_bytes()
    assert need > 0
    fake = 1 << 20                                   # never dereferenced: the checks come first
    args = [fake] * len(e.arg_shapes)
    for ws_ptr, ws_bytes in ((fake, need - 1), (fake + 8, need + 256), (0, 0)):
        with pytest.raises(TadError) as ei:
            plan.backward(args, fake, [fake] * len(args), ws_ptr, ws_bytes)
        assert ei.value.code == "TAD_ERR_WORKSPACE", (ws_ptr, ws_bytes)
    # the forward pass of the full-size workload keeps auxiliary tensors in the workspace
    big = Plan(W.FULL["cfg2"]())
    need = big.workspace_bytes()
    for ws_ptr, ws_bytes in ((fake, need - 1), (fake + 8, need + 256), (0, 0)):
        with pytest.raises(TadError) as ei:
            big.forward(args, fake, 0, ws_ptr, ws_bytes)
        assert ei.value.code == "TAD_ERR_WORKSPACE", (ws_ptr, ws_bytes)


def test_interpreter_shapes_asked_for_have_a_kernel_build():
    """The interpreter is built with bounds checks for the narrow shapes only (up to 4 values per thread, no
    element variable) and with relative loops only without an element variable; a launcher asked for anything
    else launches nothing and reports it.  The code generator must therefore never ask: every kernel header of
    debug plans and of plans with a relative loop is checked, over the reduced workloads and random expressions
    of every level."""
    from paper_1711_01348_b200 import TadError
    from workloads import configs as W
    from workloads.random_expr import random_expression

    def kernels(plan, n_access):
        for which in [-1] + list(range(n_access)) + [-2 - s for s in range(plan.num_stages())]:
            try:
                text = plan.disassemble(which)
            except TadError:
                continue
            head = None
            for line in text.splitlines():
                if line.startswith("; vars="):
                    head = dict(item.split("=") for item in line.lstrip("; ").split())
                    yield head, False
                elif line.startswith("; loop ") and " relative=1" in line and head is not None:
                    yield head, True

    exprs = [W.REDUCED[k]() for k in sorted(W.REDUCED)]
    exprs += [random_expression(seed, large=lv) for lv in (0, 1, 3, 4, 5) for seed in range(6)]
    seen_debug = seen_relative = 0
    for e in exprs:
        for debug in (False, True):
            try:
                plan = Plan(e, debug_bounds=debug)
            except TadError:
                continue
            for head, relative in kernels(plan, len(e.accesses)):
                ta, ub = (int(v.rstrip("r")) for v in head["vec"].split("x"))
                if debug:
                    assert ta <= 4 and ub == 1, head
                    seen_debug += 1
                if relative:
                    assert ub == 1, head
                    seen_relative += 1
    assert seen_debug > 50

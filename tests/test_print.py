"""tad_plan_print: the expression and its derived derivatives as text in the notation of the listing in Sec. 6.

The paper prints, for its example (a 3x5, b 4x5, c 3x3, d 8), the input expression and the four derivative
expressions; tests/golden/section6_listing.txt holds those five lines.  The printer works from the plan (Smith
normal form, kernel basis, bound rows), so agreement with the listing pins the index transform alpha = I beta + K z,
the summation ranges, the cokernel condition and the order of the chain-rule factors at once.  What is free in the
method (which of two equal indices names a position under the cokernel condition, the nesting of independent
loops, the order of the rows inside max [..] / min [..]) is normalised before comparing.  Host only."""
import os
import re

import pytest

from paper_1711_01348_b200 import Plan
from workloads import configs as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "section6_listing.txt")


def _listing():
    with open(GOLDEN) as fh:
        lines = [ln.rstrip("\n") for ln in fh if ln.strip() and not ln.startswith("#")]
    assert len(lines) == 5
    return dict(zip(["f", "da", "db", "dc", "dd"], lines))


@pytest.fixture(scope="module")
def sec6():
    e = W.intro(3, 4, 5, name="sec6")
    return e, Plan(e)


def _derivative(e, plan, name):
    arg = e.arg_names.index(name)
    qs = [q for q, a in enumerate(e.accesses) if a.arg == arg]
    assert len(qs) == 1
    return plan.print(qs[0], e.arg_names, ["i", "j", "k"])


def test_input_expression_is_printed_as_in_the_listing(sec6):
    e, plan = sec6
    assert plan.print(-1, e.arg_names, ["i", "j", "k"]) == _listing()["f"]


@pytest.mark.parametrize("name", ["a", "b"])
def test_unimodular_derivatives_match_the_listing_character_by_character(sec6, name):
    """da and db: one kernel coordinate (j resp. i), no condition; nothing is free here."""
    e, plan = sec6
    assert _derivative(e, plan, name) == _listing()["d" + name]


def test_dc_has_the_cokernel_condition_and_the_same_term(sec6):
    """c is read on its diagonal: the derivative exists where dc_0 = dc_1.  Under that condition either index
    may name the row; the listing uses dc_1, so the text is compared with dc_0 renamed inside the term."""
    e, plan = sec6
    got, want = _derivative(e, plan, "c"), _listing()["dc"]
    head = "dc[dc_0; dc_1] = if {dc_0 + -dc_1 = 0} then ("
    assert got.startswith(head) and want.startswith(head)
    assert got.endswith(") else (0)")
    assert "sum{dc_z1}_0^4 (sum{dc_z0}_0^3 (" in got                      # ranges of both kernel coordinates
    body = got[len(head):]
    renamed = re.sub(r"dc_0(?![0-9])", "dc_1", body)
    assert renamed == want[len(head):]


def _rows(text, opener):
    m = re.search(re.escape(opener) + r" \[([^\]]*)\]", text)
    assert m, (opener, text)
    return sorted(r.strip() for r in m.group(1).split(";"))


def test_dd_has_the_ranges_and_the_df_index_of_the_listing(sec6):
    """d[i + k]: two kernel coordinates; the range of the one along k depends on dd_0.  The two loops are
    independent of each other, so their nesting is free; the rows of max / min are compared as sets."""
    e, plan = sec6
    got, want = _derivative(e, plan, "d"), _listing()["dd"]
    assert "df[dd_0 + -dd_z1; dd_z0]" in got and "df[dd_0 + -dd_z1; dd_z0]" in want
    assert "sum{dd_z0}_0^3 (" in got and "sum{dd_z0}_0^3 (" in want
    assert _rows(got, "sum{dd_z1}_(max") == _rows(want, "sum{dd_z1}_(max") == ["-2 + dd_0", "0"]
    assert _rows(got, ")^(min") == _rows(want, ")^(min") == ["4", "dd_0"]
    # the term itself (everything inside the two sums) is the listing's, character by character
    term_got = got[got.index("(((-(df["):].rstrip(")")
    term_want = want[want.index("(((-(df["):].rstrip(")")
    assert term_got == term_want
    assert "if {" not in got                                                # every element of d but the last is read: no condition,


def test_divisibility_and_guards_are_printed_as_conditions():
    """y[3k] (cfg4): the derivative exists where dy_0 is a multiple of 3 (the condition the paper calls redundant
    and that is not); x of cfg3 has elements beyond the image of i + j: a guard."""
    e4 = W.REDUCED["cfg4"]()
    p4 = Plan(e4)
    dy = [p4.print(q, e4.arg_names) for q, a in enumerate(e4.accesses) if e4.arg_names[a.arg] == "y"][0]
    assert dy.startswith("dy[dy_0] = if {(dy_0) mod 3 = 0} then (") and "(1 / 3) * dy_0" in dy
    e3 = W.REDUCED["cfg3"]()
    p3 = Plan(e3)
    dx = p3.print(0, e3.arg_names)
    assert dx.startswith("dx[dx_0] = if {-600 + dx_0 <= 0} then (sum{dx_z0}_(max [")
    assert "floor ((" in p3.print(1, e3.arg_names) and "ceil ((" in p3.print(1, e3.arg_names)   # x[2i + 3j]: rows that do not divide


def test_default_names_and_missing_expressions():
    e = W.REDUCED["cfg5"]()
    p = Plan(e)
    assert p.print(-1).startswith("f[i; j; k] = sum{l}_0^12 (sum{m}_0^4 (x1[j; l; m] * x0[i; l; 2 * k + m]))")
    assert p.print(99) == ""

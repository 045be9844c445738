"""Memory model and interval chooser (Eq. 4-11, Appendix C): pinned by the closed forms, by brute force on
the integer grid, and by the constants the paper prints for three model sizes."""
import itertools
import math
import os

import pytest

from paper_2411_19460_b200 import memory_model as mm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "appendix_c_constants.txt")


def test_critical_point_zeroes_both_partials_and_gives_three_ls_two_thirds():
    for L, S in ((64, 262144), (48, 4096), (7, 30)):
        l, s, m = mm.critical_point(L, S)
        assert abs(-L * S / l ** 2 + s) < 1e-9 * s            # Eq. 5
        assert abs(-L * S / s ** 2 + l) < 1e-9 * l            # Eq. 6
        assert math.isclose(m, mm.unit_memory(L, S, l, s), rel_tol=1e-12)
        assert math.isclose(m, 3 * (L * S) ** (2 / 3), rel_tol=1e-12)   # Eq. 7
        # it is a minimum: every nearby point costs more
        for dl, ds in itertools.product((-0.01, 0, 0.01), repeat=2):
            assert mm.unit_memory(L, S, l * (1 + dl), s * (1 + ds)) >= m * (1 - 1e-12)


def test_boundary_cases_and_their_am_gm_floors():
    for L, S in ((64, 4096), (9, 100), (100, 9)):
        assert math.isclose(mm.l_bound_memory(L, S, 17), mm.unit_memory(L, S, L, 17))      # Eq. 8 is Eq. 4 at l=L
        assert math.isclose(mm.s_bound_memory(L, S, 3), mm.unit_memory(L, S, 3, S))        # Eq. 9 is Eq. 4 at s=S
        assert math.isclose(mm.l_bound_memory(L, S, math.sqrt(S)), mm.l_bound_floor(L, S))  # equality case
        assert math.isclose(mm.s_bound_memory(L, S, math.sqrt(L)), mm.s_bound_floor(L, S))
        for s in range(1, S + 1):
            assert mm.l_bound_memory(L, S, s) >= mm.l_bound_floor(L, S) - 1e-9
        for l in range(1, L + 1):
            assert mm.s_bound_memory(L, S, l) >= mm.s_bound_floor(L, S) - 1e-9


def test_regimes():
    assert mm.regime(64, 262144) == "S"           # L^2 <= S: the long-sequence case the paper trains in
    assert mm.regime(64, 4095) == "interior"
    assert mm.regime(64, 4096) == "S"
    assert mm.regime(100, 10) == "L"
    assert mm.regime(100, 11) == "interior"
    # in the interior regime the stationary point is admissible; outside, it is not
    for L, S in ((64, 4000), (30, 30)):
        l, s, _ = mm.critical_point(L, S)
        assert 1 <= l <= L and 1 <= s <= S
    l, s, _ = mm.critical_point(8, 4096)
    assert l > 8


def test_savings_ratio_grows_like_the_layer_count():
    """Eq. 11: for L^2 <= S the best integer memory is Theta(S), so L S / M* is Theta(L): here between
    L/4 and L for every tried size."""
    for L in (4, 8, 16):
        S = 4 * L * L
        best = min(mm.unit_memory(L, S, l, s) for l in range(1, L + 1) for s in range(1, S + 1))
        assert L / 4 <= L * S / best <= L


def test_constants_decode_to_the_printed_table():
    dims = {"Mamba-2-370m": 1024, "Mamba-2-1.3b": 2048, "Mamba-2-2.7b": 2560}
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for name, cl, cs, cg, cst in rows:
        c = mm.mamba2_constants(dims[name])
        assert (c.c_l, c.c_s, c.c_grid, c.c_state) == (int(cl), int(cs), int(cg), int(cst)), name


def test_estimator_terms_and_unit_model_agree():
    one = mm.MemoryConstants(1, 1, 1, 0, bytes_per_element=1)
    for L, S, l, s in ((64, 4096, 4, 64), (12, 100, 5, 10)):
        est = mm.expected_memory(L, S, l, s, one)
        assert math.isclose(est.total, mm.unit_memory(L, S, l, s))
    c = mm.mamba2_constants(2560)
    est = mm.expected_memory(64, 1 << 19, 8, 4096, c)
    assert est.l_ckpt == 64 * (1 << 19) / 8 * 2560 * 2
    assert est.s_ckpt == 64 * (1 << 19) / 4096 * 671488 * 2
    assert est.grid == 8 * 4096 * 15696 * 2
    assert est.state == 4096 * 660736 * 2


def test_chooser_equals_brute_force_and_respects_budget():
    c = mm.mamba2_constants(1024)
    for L, S, mult in ((6, 96, 8), (5, 64, 1), (12, 256, 16)):
        l, s, est = mm.choose_intervals(L, S, c, seg_multiple=mult)
        brute = min((mm.expected_memory(L, S, a, b, c).total, a, -b)
                    for a in range(1, L + 1) for b in range(mult, S + 1, mult) if S % b == 0)
        assert (est.total, l, -s) == brute
        # continuous optimum is a lower bound for the integer one, and close to it
        _, _, m_cont = mm.continuous_optimum(L, S, c)
        assert m_cont <= est.total * (1 + 1e-12)
    # budget: least recomputation that fits
    L, S = 12, 256
    full = mm.expected_memory(L, S, 1, S, c).total
    l, s, est = mm.choose_intervals(L, S, c, seg_multiple=16, budget_bytes=full)
    assert l == 1 and est.total <= full
    tight = mm.choose_intervals(L, S, c, seg_multiple=16)[2].total
    l2, s2, est2 = mm.choose_intervals(L, S, c, seg_multiple=16, budget_bytes=tight)
    assert est2.total <= tight
    assert mm.choose_intervals(L, S, c, seg_multiple=16, budget_bytes=tight * 0.99) is None


def test_continuous_optimum_is_stationary():
    c = mm.mamba2_constants(2560)
    L, S = 64, 1 << 19
    l, s, m = mm.continuous_optimum(L, S, c)
    assert 1 < l < L and 1 < s < S
    e = 1e-6
    f = lambda a, b: mm.expected_memory(L, S, a, b, c).total
    assert abs(f(l * (1 + e), s) - f(l * (1 - e), s)) / (2 * e * m) < 1e-6
    assert abs(f(l, s * (1 + e)) - f(l, s * (1 - e))) / (2 * e * m) < 1e-6
    # the paper reports 42.2 GB of activations at this length for this model: the estimate at the
    # optimum is of that order (a sanity range, not a pin: the measured figure includes the allocator)
    assert 10e9 < m < 42.2e9


def test_layer_stack_bytes_formula():
    b = mm.layer_stack_bytes(64, 262144, 2, 4096, 80, 64, 128)
    assert b["layer_inputs"] == 33 * 262144 * 80 * 64 * 2
    assert b["boundary_states"] == 64 * 65 * 80 * 64 * 128 * 4
    assert b["cell_inputs"] == 4096 * 80 * 64 * 2
    b = mm.layer_stack_bytes(4, 1024, 3, 256, 4, 64, 128)
    assert b["layer_inputs"] == 3 * 1024 * 4 * 64 * 2          # x0, x3, x4

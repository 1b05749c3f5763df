"""Pins for the controller half of the CPU oracle: cost lookup, cumulative maximum, exhaustive Eq. (1)."""
from pathlib import Path

import numpy as np
import pytest

GOLDEN = Path(__file__).resolve().parent / "golden"
MS = 1_000_000


def read_rows(name):
    rows = []
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append([int(x) for x in line.split()])
    return rows


# ------------------------------------------------------------------------------------------------
# closed form under the analytic model (Sec. 4.1) — golden values worked out by hand
# ------------------------------------------------------------------------------------------------
def test_analytic_cost_printed_coefficients(oracle):
    assert oracle.analytic_cost_ns(0, 0) == 350_000
    assert oracle.analytic_cost_ns(1, 0) == 350_000 + 900_000 + 55_000
    assert oracle.analytic_cost_ns(0, 1) == 350_000 + 400_000 + 6_000
    assert oracle.analytic_cost_ns(64, 3305) == 25 * MS  # exact tie used by the golden file
    assert oracle.analytic_cost_ns(10, 100) == 350_000 + 900_000 + 550_000 + 400_000 + 600_000


@pytest.mark.parametrize("row", read_rows("analytic_model_chunks.txt"))
def test_bruteforce_matches_closed_form_golden(oracle, row):
    n, budget, L, want_chunk, want_infeasible = row
    table = oracle.analytic_table([n], 4096)
    now = 123_456_789
    deadlines = np.full(n, now + budget + 5 * MS, dtype=np.int64)
    deadlines[n // 2] = now + budget  # the earliest one decides
    chunk, flags, B = table.choose(now, deadlines, total_ctx=n * 1000, prefix_len=0, remaining=L, c_max=4096)
    assert B == budget
    assert chunk == want_chunk
    assert bool(flags & oracle.F_DECODE_INFEASIBLE) == bool(want_infeasible)
    # the closed form itself
    t0 = 350_000 + 900_000 + 55_000 * n
    closed = min(L, (budget - t0 - 400_000) // 6000) if budget - t0 - 400_000 >= 6000 else 0
    assert chunk == closed


def test_eq1_set_definition_on_analytic_model(oracle):
    """chunk == max of the feasible set written as a python set comprehension."""
    def T(n, c):
        return 350_000 + (900_000 + 55_000 * n if n else 0) + (400_000 + 6_000 * c if c else 0)

    table = oracle.analytic_table([1, 8, 32, 100], 600)
    rng = np.random.default_rng(0)
    for _ in range(300):
        n = int(rng.choice([1, 8, 32, 100]))
        L = int(rng.integers(1, 601))
        budget = int(rng.integers(0, 12 * MS))
        feas = {c for c in range(0, L + 1) if T(n, c) <= budget}
        want = max(feas) if feas else 0
        chunk, flags, _ = table.choose(0, [budget] * n, n, 0, L, c_max=600)
        assert chunk == want
        assert bool(flags & oracle.F_DECODE_INFEASIBLE) == (T(n, 0) > budget)


# ------------------------------------------------------------------------------------------------
# branch cases of Algorithm 1 / Sec. 3.1
# ------------------------------------------------------------------------------------------------
def test_branch_cases(oracle):
    table = oracle.analytic_table([4], 4096)
    now = 10 * MS
    dl = [now + 25 * MS] * 4
    # no pending prefill
    assert table.choose(now, dl, 4, 0, 0)[:2] == (0, oracle.F_NO_PREFILL)
    # no active decode: L = min(C_max, remaining), table never consulted (out-of-grid n would raise)
    assert table.choose(now, [], 10**15, 10**9, 9000, c_max=4096)[:2] == (4096, oracle.F_NO_DECODE | oracle.F_CAPPED)
    assert table.choose(now, [], 0, 0, 100, c_max=4096)[:2] == (100, oracle.F_NO_DECODE)
    # deadline already past -> budget clamps to 0 -> nothing fits, decode-only is itself late
    c, f, B = table.choose(now, [now - 5] * 4, 4, 0, 512)
    assert (c, B) == (0, 0) and f & oracle.F_DECODE_INFEASIBLE
    # huge budget recovers the full remaining prompt (full prefill when it fits)
    assert table.choose(now, [now + 10**12] * 4, 4, 0, 3000)[0] == 3000
    # feasibility is non-strict: a tie is feasible, one ns less is not
    t = oracle.analytic_cost_ns(4, 100)
    assert table.choose(0, [t] * 4, 4, 0, 4096)[0] == 100
    assert table.choose(0, [t - 1] * 4, 4, 0, 4096)[0] == 99


def test_heterogeneous_deadlines(oracle):
    table = oracle.analytic_table([6], 2048)
    rng = np.random.default_rng(3)
    dl = rng.integers(5 * MS, 30 * MS, size=6).astype(np.int64)
    base = table.choose(0, dl, 6, 0, 2048, c_max=2048)[0]
    for _ in range(5):
        assert table.choose(0, rng.permutation(dl), 6, 0, 2048, c_max=2048)[0] == base
    for i in range(6):
        tight = dl.copy()
        tight[i] -= 2 * MS
        assert table.choose(0, tight, 6, 0, 2048, c_max=2048)[0] <= base


def test_margin_and_quantum(oracle):
    table = oracle.analytic_table([8], 1024)
    budget = 6 * MS
    plain = table.choose(0, [budget] * 8, 8, 0, 1024, c_max=1024)[0]
    t0 = 350_000 + 900_000 + 55_000 * 8 + 400_000
    assert plain == (budget - t0) // 6000
    # absolute margin shifts the budget
    assert table.choose(0, [budget] * 8, 8, 0, 1024, c_max=1024, margin_abs_ns=600_000)[0] == (budget - 600_000 - t0) // 6000
    # relative margin: T * 1.05 <= B, checked through the set definition
    def T(c):
        return t0 - 400_000 + (400_000 + 6000 * c if c else 0)
    want = max(c for c in range(0, 1025) if T(c) + -(-T(c) * 50_000 // 1_000_000) <= budget)
    assert table.choose(0, [budget] * 8, 8, 0, 1024, c_max=1024, margin_ppm=50_000)[0] == want
    # quantum: only multiples of 16 that are <= L
    assert table.choose(0, [budget] * 8, 8, 0, 1024, c_max=1024, quantum=16)[0] == plain // 16 * 16
    assert table.choose(0, [10**12] * 8, 8, 0, 100, c_max=1024, quantum=16)[0] == 96


# ------------------------------------------------------------------------------------------------
# lookup: ceil-step rounding, optional interpolation, out-of-grid behaviour — worked numbers
# ------------------------------------------------------------------------------------------------
def test_lookup_ceil_step_and_interpolation(oracle):
    cost = np.arange(2 * 2 * 2 * 3, dtype=np.int64).reshape(2, 2, 2, 3) * 100 + 1000
    t = oracle.Table([4, 16], [1000, 8000], [0, 4096], [0, 64, 256], cost)
    assert t.lookup(4, 1000, 0, 0) == cost[0, 0, 0, 0]
    assert t.lookup(16, 8000, 4096, 256) == cost[1, 1, 1, 2]
    assert t.lookup(1, 1, 0, 1) == cost[0, 0, 0, 1]          # everything rounds up
    assert t.lookup(5, 1001, 1, 65) == cost[1, 1, 1, 2]
    assert t.lookup(4, 1000, 0, 257) == oracle.INF            # chunk beyond the grid is infeasible
    for bad in ((17, 1, 0, 1), (1, 8001, 0, 1), (1, 1, 4097, 1)):
        with pytest.raises(IndexError):
            t.lookup(*bad)
    ti = oracle.Table([4], [1000], [0], [0, 64, 256], [[[[1000, 2000, 2960]]]], interp=True)
    assert ti.lookup(4, 1000, 0, 64) == 2000
    assert ti.lookup(4, 1000, 0, 32) == 1500                  # halfway 1000..2000
    assert ti.lookup(4, 1000, 0, 65) == 2005                  # 2000 + ceil(960*1/192) = 2000 + 5
    assert ti.lookup(4, 1000, 0, 255) == 2955
    assert ti.lookup(4, 1000, 0, 1) == 1000 + 16              # ceil(1000/64) = 16


def test_cummax_worked_example(oracle):
    rows = read_rows("cummax_worked_example.txt")
    grid, raw, mono = rows[0], rows[1], rows[2]
    t_raw = oracle.Table([1], [10], [0], grid, raw)
    t_mono = oracle.Table([1], [10], [0], grid, raw).cummax()
    assert t_mono.cost.reshape(-1).tolist() == mono
    for budget, want_raw, want_mono in rows[3:]:
        assert t_raw.choose(0, [budget], 10, 0, 112, c_max=112)[0] == want_raw
        assert t_mono.choose(0, [budget], 10, 0, 112, c_max=112)[0] == want_mono


def test_cummax_all_axes(oracle):
    rng = np.random.default_rng(1)
    cost = rng.integers(1, 1000, size=(3, 4, 2, 5)).astype(np.int64)
    t = oracle.Table([1, 2, 3], [1, 2, 3, 4], [0, 1], [0, 1, 2, 3, 4], cost).cummax()
    c = t.cost
    for ax in range(4):
        assert np.all(np.diff(c, axis=ax) >= 0)
    assert np.all(c >= cost)
    # minimality on the chunk axis for the first line: plain running maximum
    assert np.array_equal(c[0, 0, 0], np.maximum.accumulate(cost[0, 0, 0]))


def test_maximality_property_on_random_monotone_tables(oracle):
    """Proposition 1: the scan's answer is feasible and the next candidate is not."""
    rng = np.random.default_rng(7)
    for trial in range(40):
        nk = int(rng.integers(2, 12))
        grid = np.cumsum(rng.integers(1, 40, size=nk)).astype(np.int32)
        grid[0] = 0 if trial % 2 == 0 else grid[0]
        cost = np.cumsum(rng.integers(0, 500, size=nk)).astype(np.int64) + 100
        t = oracle.Table([8], [100], [0], grid, cost, interp=bool(trial % 3 == 0))
        L = int(rng.integers(1, int(grid[-1]) + 20))
        for budget in sorted(set([0, 99, 100] + [int(x) + d for x in cost for d in (-1, 0, 1)])):
            c, flags, _ = t.choose(0, [budget] * 8, 100, 0, L, c_max=10**6)
            assert 0 <= c <= L
            if c > 0:
                assert t.lookup(8, 100, 0, c) <= budget
            if c < L:
                assert t.lookup(8, 100, 0, c + 1) > budget
            assert bool(flags & oracle.F_DECODE_INFEASIBLE) == (t.lookup(8, 100, 0, 0) > budget)

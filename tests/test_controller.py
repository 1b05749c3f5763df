"""sw_choose_chunk (Algorithm 1, bisection) against the oracle's exhaustive Eq. (1) scan: bit-exact."""
from pathlib import Path

import numpy as np
import pytest

MS = 1_000_000
GOLDEN = Path(__file__).resolve().parent / "golden"


@pytest.fixture(scope="module")
def B():
    from paper_2609_07883_b200 import build

    build.build()
    from paper_2609_07883_b200 import binding

    return binding


def both_tables(B, oracle, n_grid, ctx_grid, prefix_grid, chunk_grid, cost, interp=False, monotone=True):
    lib_t = B.CostTable(n_grid, ctx_grid, prefix_grid, chunk_grid, cost, make_monotone=monotone, interp=interp)
    ora_t = oracle.Table(n_grid, ctx_grid, prefix_grid, chunk_grid, cost, interp=interp)
    if monotone:
        ora_t.cummax()
    return lib_t, ora_t


def random_table(rng, monotone_input):
    nn, nc, np_ = (int(rng.integers(1, 4)) for _ in range(3))
    nk = int(rng.integers(2, 10))
    n_grid = np.cumsum(rng.integers(1, 50, size=nn))
    ctx_grid = np.cumsum(rng.integers(1, 10**6, size=nc)).astype(np.int64)
    prefix_grid = np.cumsum(rng.integers(0, 5000, size=np_)) + np.arange(np_)
    chunk_grid = np.cumsum(rng.integers(1, 300, size=nk))
    if rng.integers(0, 2):
        chunk_grid[0] = 0
    cost = rng.integers(50_000, 30 * MS, size=(nn, nc, np_, nk)).astype(np.int64)
    if monotone_input:
        for ax in range(4):
            cost = np.maximum.accumulate(cost, axis=ax)
    return n_grid, ctx_grid, prefix_grid, chunk_grid, cost


def test_tables_agree_with_oracle_lookup(B, oracle):
    rng = np.random.default_rng(100)
    for trial in range(30):
        grids = random_table(rng, monotone_input=False)
        interp = bool(trial % 2)
        lt, ot = both_tables(B, oracle, *grids, interp=interp)
        n_grid, ctx_grid, prefix_grid, chunk_grid, _ = grids
        for _ in range(200):
            n = int(rng.integers(0, n_grid[-1] + 1))
            ctx = int(rng.integers(0, ctx_grid[-1] + 1))
            pre = int(rng.integers(0, prefix_grid[-1] + 1))
            c = int(rng.integers(0, chunk_grid[-1] + 40))
            assert lt.lookup(n, ctx, pre, c) == ot.lookup(n, ctx, pre, c)
        with pytest.raises(B.SwError) as e:
            lt.lookup(int(n_grid[-1]) + 1, 0, 0, 0)
        assert e.value.status == B.SW_ERR_OUT_OF_RANGE


@pytest.mark.parametrize("interp", [False, True])
def test_bisection_equals_exhaustive_scan_on_random_monotone_tables(B, oracle, interp):
    rng = np.random.default_rng(200 + int(interp))
    for trial in range(60):
        grids = random_table(rng, monotone_input=bool(trial % 2))
        lt, ot = both_tables(B, oracle, *grids, interp=interp)
        n_grid, ctx_grid, prefix_grid, chunk_grid, _ = grids
        values = sorted(set(int(v) for v in ot.cost.reshape(-1)))
        budgets = [0, 1] + [v + d for v in values[:: max(1, len(values) // 12)] for d in (-1, 0, 1)] + [10**12]
        for budget in budgets:
            n = int(rng.integers(1, n_grid[-1] + 1))
            ctx = int(rng.integers(0, ctx_grid[-1] + 1))
            pre = int(rng.integers(0, prefix_grid[-1] + 1))
            remaining = int(rng.integers(1, chunk_grid[-1] + 60))
            c_max = int(rng.choice([64, 512, 4096]))
            quantum = int(rng.choice([1, 1, 16]))
            ppm = int(rng.choice([0, 50_000]))
            mabs = int(rng.choice([0, 12_345]))
            now = int(rng.integers(0, 10**9))
            dl = now + budget + rng.integers(0, 5 * MS, size=n)
            dl[rng.integers(0, n)] = now + budget
            got = B.sw_choose_chunk(lt, now, dl, ctx, pre, remaining, c_max=c_max, chunk_quantum=quantum,
                                    margin_abs_ns=mabs, margin_ppm=ppm)
            want = ot.choose(now, dl, ctx, pre, remaining, c_max=c_max, quantum=quantum, margin_abs_ns=mabs,
                             margin_ppm=ppm)
            assert (got.chunk, got.flags, got.budget_ns) == want, (trial, budget)
            L = min(c_max, remaining) // quantum
            assert got.queries <= max(1, int(np.ceil(np.log2(L + 1)))) if L > 0 else got.queries == 0


def test_branch_cases_and_flags(B, oracle):
    table = oracle.analytic_table([4], 4096)
    lt = B.CostTable(table.n_grid, table.ctx_grid, table.prefix_grid, table.chunk_grid, table.cost)
    now = 10 * MS
    dl = np.array([now + 25 * MS] * 4)
    r = B.sw_choose_chunk(lt, now, dl, 4, 0, 0)
    assert (r.chunk, r.flags, r.queries) == (0, B.SW_F_NO_PREFILL, 0)
    r = B.sw_choose_chunk(None, now, [], 10**15, 10**9, 9000, c_max=4096)      # no table needed without decodes
    assert (r.chunk, r.flags, r.queries) == (4096, B.SW_F_NO_DECODE | B.SW_F_CAPPED, 0)
    r = B.sw_choose_chunk(lt, now, dl - 40 * MS, 4, 0, 512)
    assert r.chunk == 0 and r.budget_ns == 0 and r.flags & B.SW_F_DECODE_INFEASIBLE
    r = B.sw_choose_chunk(lt, now, dl + 10**12, 4, 0, 3000)
    assert r.chunk == 3000 and r.flags == 0
    t = oracle.analytic_cost_ns(4, 100)
    assert B.sw_choose_chunk(lt, 0, [t] * 4, 4, 0, 4096).chunk == 100
    assert B.sw_choose_chunk(lt, 0, [t] * 4, 4, 0, 4096).predicted_ns == t
    assert B.sw_choose_chunk(lt, 0, [t - 1] * 4, 4, 0, 4096).chunk == 99
    with pytest.raises(B.SwError) as e:
        B.sw_choose_chunk(lt, 0, [t] * 5, 5, 0, 4096)     # n = 5 beyond the table's n grid
    assert e.value.status == B.SW_ERR_OUT_OF_RANGE


def test_golden_closed_form_chunks(B, oracle):
    for line in (GOLDEN / "analytic_model_chunks.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        n, budget, L, want_chunk, want_inf = (int(x) for x in line.split())
        table = oracle.analytic_table([n], 4096)
        lt = B.CostTable(table.n_grid, table.ctx_grid, table.prefix_grid, table.chunk_grid, table.cost)
        r = B.sw_choose_chunk(lt, 7, [7 + budget] * n, n * 500, 0, L, c_max=4096)
        assert r.chunk == want_chunk
        assert bool(r.flags & B.SW_F_DECODE_INFEASIBLE) == bool(want_inf)


def test_raw_non_monotone_table_breaks_bisection_and_cummax_restores_it(B, oracle):
    rows = [[int(x) for x in l.split()] for l in (GOLDEN / "cummax_worked_example.txt").read_text().splitlines()
            if l.strip() and not l.startswith("#")]
    grid, raw = rows[0], rows[1]
    with pytest.raises(B.SwError) as e:
        B.CostTable([1], [10], [0], grid, raw, make_monotone=False)
    assert e.value.status == B.SW_ERR_NOT_MONOTONE
    lt = B.CostTable([1], [10], [0], grid, raw, make_monotone=True)
    for budget, _want_raw, want_mono in rows[3:]:
        assert B.sw_choose_chunk(lt, 0, [budget], 10, 0, 112, c_max=112).chunk == want_mono


def test_first_fit_over_several_pending_requests_matches_the_oracle(B, oracle):
    """sw_choose_chunks against the oracle's exhaustive scan on random monotone tables (bit-exact lists and budget)."""
    rng = np.random.default_rng(21)
    for trial in range(12):
        grids = random_table(rng, monotone_input=False)
        lt, ot = both_tables(B, oracle, *grids)
        n_grid, ctx_grid, prefix_grid, chunk_grid, _ = grids
        values = sorted(set(int(v) for v in ot.cost.reshape(-1)))
        for _ in range(40):
            n = int(rng.integers(0, n_grid[-1] + 1))
            ctx = int(rng.integers(0, ctx_grid[-1] + 1))
            m = int(rng.integers(1, 11))
            # keep the summed prefixes inside the table's prefix axis
            prefixes = [int(x) for x in rng.integers(0, max(1, int(prefix_grid[-1]) // 10) + 1, size=m)]
            remaining = [int(x) for x in rng.integers(1, int(chunk_grid[-1]) + 50, size=m)]
            c_max = int(rng.integers(1, int(chunk_grid[-1]) + 100))
            quantum = int(rng.choice([1, 1, 16]))
            now = int(rng.integers(0, 10**6))
            budget = int(rng.choice(values)) + int(rng.integers(-2, 3)) if rng.integers(0, 4) else int(rng.integers(0, 10**12))
            dl = now + max(0, budget) + rng.integers(0, 5 * MS, size=n)
            if n:
                dl[rng.integers(0, n)] = now + max(0, budget)
            mabs, mppm = int(rng.integers(0, 1000)), int(rng.choice([0, 50_000]))
            got, ch = B.sw_choose_chunks(lt if n else None, now, dl, ctx, prefixes, remaining, c_max=c_max,
                                         chunk_quantum=quantum, margin_abs_ns=mabs, margin_ppm=mppm)
            want, want_budget = oracle.choose_first_fit(ot, now, dl, ctx, prefixes, remaining, c_max=c_max, quantum=quantum,
                                                        margin_abs_ns=mabs, margin_ppm=mppm)
            assert got == want, (trial, n, prefixes, remaining, c_max, quantum, budget)
            assert ch.chunk == sum(want) and ch.budget_ns == want_budget
            if m == 1 and n > 0:
                one = B.sw_choose_chunk(lt, now, dl, ctx, prefixes[0], remaining[0], c_max=c_max, chunk_quantum=quantum,
                                        margin_abs_ns=mabs, margin_ppm=mppm)
                assert ([one.chunk] if one.chunk else []) == got and one.predicted_ns == ch.predicted_ns


def test_decode_only_cost_is_read_at_prefix_zero(B, oracle):
    """A table whose c = 0 column differs between prefix points: an iteration without prefill tokens processes no prompt,
    so both entry points (and the exhaustive scan) decide SW_F_DECODE_INFEASIBLE by the cost at prefix 0, and agree."""
    grids = ([4], [1000], [0, 100], [0, 16], np.array([10, 20, 50, 60], dtype=np.int64))
    lt, ot = both_tables(B, oracle, *grids)
    one = B.sw_choose_chunk(lt, 0, [30] * 4, 1000, 100, 64)
    many, ch = B.sw_choose_chunks(lt, 0, [30] * 4, 1000, [100], [64])
    want = ot.choose(0, [30] * 4, 1000, 100, 64)
    assert want == (0, 0, 30)
    assert (one.chunk, one.flags, one.budget_ns, one.predicted_ns) == (0, 0, 30, 10)
    assert many == [] and (ch.chunk, ch.flags, ch.budget_ns, ch.predicted_ns) == (0, 0, 30, 10)
    # at prefix 0 the 16-token chunk costs 20 and fits; at prefix 100 it costs 60 and does not
    assert B.sw_choose_chunk(lt, 0, [30] * 4, 1000, 0, 64).chunk == 16
    # below the decode-only cost the flag is raised, by all three
    assert B.sw_choose_chunk(lt, 0, [9] * 4, 1000, 100, 64).flags == B.SW_F_DECODE_INFEASIBLE
    assert B.sw_choose_chunks(lt, 0, [9] * 4, 1000, [100], [64])[1].flags == B.SW_F_DECODE_INFEASIBLE
    assert ot.choose(0, [9] * 4, 1000, 100, 64) == (0, B.SW_F_DECODE_INFEASIBLE, 9)

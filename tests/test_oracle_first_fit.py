"""Pins of the oracle's first-fit chooser for several prefills per iteration (Sec. 3.3, "Prefill batching")."""
import numpy as np

from oracle import sw_oracle as O

MS = 1_000_000


def table(n_values=(1, 4, 8, 16), c_max=1024):
    return O.analytic_table(n_values, c_max)


def test_one_pending_request_is_algorithm_1():
    t = table()
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.choice([1, 4, 8, 16]))
        budget = int(rng.integers(0, 12 * MS))
        remaining = int(rng.integers(1, 1500))
        q = int(rng.choice([1, 16]))
        single = t.choose(0, [budget] * n, 100, 0, remaining, c_max=1024, quantum=q)
        many, b = O.choose_first_fit(t, 0, [budget] * n, 100, [0], [remaining], c_max=1024, quantum=q)
        assert b == single[2]
        assert many == ([single[0]] if single[0] > 0 else [])


def test_closed_form_with_the_analytic_model():
    # T(n, c) = 0.35 + 0.90 + 0.055 n + 0.40 + 0.006 c ms: with n = 4 and B = 5 ms the token budget is
    # floor((5 - 1.87) / 0.006) = 521 tokens in total, whatever the number of requests they come from
    t = table()
    chunks, b = O.choose_first_fit(t, 0, [5 * MS] * 4, 100, [0, 0, 0, 0], [100, 200, 300, 400], c_max=1024)
    assert b == 5 * MS
    assert chunks == [100, 200, 221]                  # two whole prompts, the third cut, the fourth not looked at
    # a budget that fits everything admits every request whole
    chunks, _ = O.choose_first_fit(t, 0, [50 * MS] * 4, 100, [0, 0, 0], [100, 200, 300], c_max=1024)
    assert chunks == [100, 200, 300]
    # C_max caps the total
    chunks, _ = O.choose_first_fit(t, 0, [50 * MS] * 4, 100, [0, 0, 0], [100, 200, 300], c_max=256)
    assert chunks == [100, 156]
    # not even one token fits: nothing is admitted
    chunks, _ = O.choose_first_fit(t, 0, [1 * MS] * 4, 100, [0, 0], [100, 200], c_max=1024)
    assert chunks == []
    # no active decode: no deadline, whole requests up to C_max, at most max_chunks of them
    chunks, b = O.choose_first_fit(t, 0, [], 0, [0] * 10, [50] * 10, c_max=1024, max_chunks=8)
    assert b == 0 and chunks == [50] * 8
    # quantum: a cut chunk is a multiple of it
    chunks, _ = O.choose_first_fit(t, 0, [5 * MS] * 4, 100, [0, 0], [96, 800], c_max=1024, quantum=16)
    assert chunks == [96, 416]                        # 521 - 96 = 425 -> 416


def test_every_admitted_list_fits_and_the_next_token_would_not():
    """Properties that hold for any monotone table: the total fits the budget; one quantum more on the last admitted
    request (if it was cut) does not."""
    rng = np.random.default_rng(1)
    n_grid, ctx_grid, prefix_grid = [1, 8], [1000], [0, 512, 2048, 8192]
    chunk_grid = list(range(0, 1025, 16))
    raw = rng.integers(1, 40_000, size=(2, 1, 4, len(chunk_grid))).astype(np.int64)
    t = O.Table(n_grid, ctx_grid, prefix_grid, chunk_grid, raw).cummax()
    for _ in range(150):
        n = int(rng.choice([1, 8]))
        budget = int(rng.integers(0, int(t.cost.max()) + 1000))
        m = int(rng.integers(1, 5))
        prefixes = [int(x) for x in rng.integers(0, 2000, size=m)]
        remaining = [int(x) for x in rng.integers(1, 600, size=m)]
        chunks, b = O.choose_first_fit(t, 0, [budget] * n, 500, prefixes, remaining, c_max=1024)
        assert len(chunks) <= m and all(0 < c <= r for c, r in zip(chunks, remaining))
        assert all(c == r for c, r in zip(chunks[:-1], remaining))      # only the last one may be cut
        if chunks:
            assert t.lookup(n, 500, sum(prefixes[:len(chunks)]), sum(chunks)) <= b
            if chunks[-1] < remaining[len(chunks) - 1] and sum(chunks) < 1024:
                assert t.lookup(n, 500, sum(prefixes[:len(chunks)]), sum(chunks) + 1) > b

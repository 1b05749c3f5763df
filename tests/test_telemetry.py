"""The library's residual table against the oracle's plain definition (bit-exact), its argument checks, and the
feedback loop on the CPU: a cost model that under-predicts, with and without the residual margin."""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W


@pytest.fixture(scope="module")
def B():
    from paper_2609_07883_b200 import build

    build.build()
    from paper_2609_07883_b200 import binding

    return binding


def test_margins_match_the_oracle_on_random_streams(B, oracle):
    rng = np.random.default_rng(11)
    for trial in range(6):
        n_edges = sorted(set(int(x) for x in rng.integers(1, 600, size=int(rng.integers(1, 6)))))
        c_edges = sorted(set([0] + [int(x) for x in rng.integers(1, 5000, size=int(rng.integers(1, 6)))]))
        window = int(rng.integers(1, 40))
        lib_t = B.Telemetry(n_edges, c_edges, window)
        ref_t = oracle.ResidualTable(n_edges, c_edges, window)
        for step in range(400):
            n, c = int(rng.integers(0, 700)), int(rng.integers(0, 6000))
            pred, obs = int(rng.integers(0, 10**7)), int(rng.integers(0, 10**7))
            lib_t.record(n, c, pred, obs, slack_ns=int(rng.integers(-5, 5)), fallback=bool(step % 7 == 0))
            ref_t.record(n, c, pred, obs)
            if step == 250 and trial % 2:
                lib_t.reset()
                ref_t.reset()
            if step % 9 == 0:
                qn, qc = int(rng.integers(0, 700)), int(rng.integers(0, 6000))
                ppm = int(rng.choice([1, 500_000, 900_000, 990_000, 1_000_000]))
                ms, fl = int(rng.integers(1, 6)), int(rng.integers(0, 1000))
                assert lib_t.margin(qn, qc, ppm, ms, fl) == ref_t.margin(qn, qc, ppm, ms, fl)
                cfg = int(rng.integers(0, 10**7))
                assert lib_t.exceeds(qn, qc, cfg, ppm, ms) == ref_t.exceeds(qn, qc, cfg, ppm, ms)
        tot = lib_t.totals()
        assert tot["records"] == 400 == ref_t.records
        assert tot["fallbacks"] == len(range(0, 400, 7))


def test_totals_and_argument_checks(B):
    t = B.Telemetry([8], [0, 4096], window=4)
    t.record(3, 100, 1000, 1500, slack_ns=-1)
    t.record(3, 100, 1000, 900, slack_ns=10, fallback=True)
    assert t.totals() == {"records": 2, "fallbacks": 1, "deadline_misses": 1, "max_residual_ns": 500}
    with pytest.raises(B.SwError):
        B.Telemetry([8, 8], [0], window=4)             # edges must increase strictly
    with pytest.raises(B.SwError):
        B.Telemetry([8], [0], window=0)
    with pytest.raises(B.SwError):
        t.margin(1, 1, percentile_ppm=0)
    with pytest.raises(B.SwError):
        t.record(-1, 0, 0, 0)


def test_feedback_loop_absorbs_an_under_predicting_table(B, oracle):
    """The executor is 12 % slower than the table says.  Open loop, the controller fills the budget with its own
    prediction and misses deadlines; with the residual margin fed back it stops missing after the warm-up, and the
    fallback rule fires while the residuals are above the configured margin."""
    from paper_2609_07883_b200 import serving

    n_values = list(range(1, 129))
    chunk_grid = list(range(0, 2049, 16))
    cost = np.array([[oracle.analytic_cost_ns(n, c) for c in chunk_grid] for n in n_values], dtype=np.int64)
    table = B.CostTable(n_values, [1 << 40], [1 << 30], chunk_grid, cost.reshape(len(n_values), 1, 1, -1))
    trace = W.bursty_trace(num_requests=300, rate_low=30.0, rate_high=90.0, mean_dwell_s=1.0, prompt_median=1500.0,
                           prompt_clip=(32, 4096), mean_output=60.0, rng=np.random.default_rng(9))

    def slow(batch):
        return int(oracle.analytic_cost_ns(batch.num_decode, batch.chunk_len) * 1.12)

    kw = dict(shape=W.LLAMA, num_pages=1 << 16, policy="sloweave", c_max=2048, margin_ppm=0, quantum=16, max_decode=128,
              page_tables=False)
    open_loop = serving.run_trace(trace, 10.0, table, slow, **kw)
    assert open_loop["deadline_misses_with_chunk"] > 20
    tel = B.Telemetry([4, 16, 64, 128], [0, 256, 1024, 2048], window=128)
    closed = serving.run_trace(trace, 10.0, table, slow, telemetry=tel, fallback_margin_ns=5_000_000, **kw)
    assert closed["deadline_misses_with_chunk"] <= open_loop["deadline_misses_with_chunk"] // 10
    assert closed["prefill_tokens"] == open_loop["prefill_tokens"] == int(trace["prompt_len"].sum())
    tot = tel.totals()
    # iterations with at least one active decode are recorded (the rest have no deadline to predict against)
    assert 0.9 * closed["iterations"] < tot["records"] <= closed["iterations"]
    assert closed["fallback_iterations"] == tot["fallbacks"]
    # a configured margin below the residuals (12 % of a 10 ms iteration is 1.2 ms) makes the fallback rule fire
    tel2 = B.Telemetry([4, 16, 64, 128], [0, 256, 1024, 2048], window=128)
    strict = serving.run_trace(trace, 10.0, table, slow, telemetry=tel2, fallback_margin_ns=200_000, **kw)
    assert strict["fallback_iterations"] > 0
    assert strict["prefill_tokens"] == int(trace["prompt_len"].sum())


def test_reprofiling_hook_replaces_a_stale_table(B, oracle):
    """Sec. 5.1: when the residuals keep exceeding the configured margin the runtime measures a new table.  Here the
    executor is 12 % slower than the first table; the hook returns a table of the slower machine, after which the
    fallback stops firing."""
    from paper_2609_07883_b200 import serving

    n_values = list(range(1, 129))
    chunk_grid = list(range(0, 2049, 16))
    cost = np.array([[oracle.analytic_cost_ns(n, c) for c in chunk_grid] for n in n_values], dtype=np.int64)
    stale = B.CostTable(n_values, [1 << 40], [1 << 30], chunk_grid, cost.reshape(len(n_values), 1, 1, -1))
    fresh_cost = (cost * 1.12).astype(np.int64) + 1
    calls = []

    def reprofile():
        calls.append(1)
        return B.CostTable(n_values, [1 << 40], [1 << 30], chunk_grid, fresh_cost.reshape(len(n_values), 1, 1, -1))

    trace = W.bursty_trace(num_requests=300, rate_low=30.0, rate_high=90.0, mean_dwell_s=1.0, prompt_median=1500.0,
                           prompt_clip=(32, 4096), mean_output=60.0, rng=np.random.default_rng(9))
    slow = lambda batch: int(oracle.analytic_cost_ns(batch.num_decode, batch.chunk_len) * 1.12)
    kw = dict(shape=W.LLAMA, num_pages=1 << 16, policy="sloweave", c_max=2048, margin_ppm=0, quantum=16, max_decode=128,
              page_tables=False, fallback_margin_ns=200_000)
    tel = B.Telemetry([4, 16, 64, 128], [0, 256, 1024, 2048], window=32)
    without = serving.run_trace(trace, 10.0, stale, slow, telemetry=B.Telemetry([4, 16, 64, 128], [0, 256, 1024, 2048], window=32),
                                **kw)
    with_hook = serving.run_trace(trace, 10.0, stale, slow, telemetry=tel, reprofile=reprofile, reprofile_after_fallbacks=32,
                                  **kw)
    assert len(calls) == with_hook["reprofiles"] >= 1
    assert with_hook["fallback_iterations"] < without["fallback_iterations"] // 4
    assert with_hook["prefill_tokens"] == int(trace["prompt_len"].sum())

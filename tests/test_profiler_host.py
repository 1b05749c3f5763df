"""Host-side pieces of the measurement path that need no GPU: the sample-size rule of the cost-table profiler, the report on
what the cumulative maximum raised, and the clock record of a timed window."""
import numpy as np
import pytest


def test_sample_size_rule():
    from paper_2609_07883_b200 import profiler

    assert profiler.reps_for(999_999) == 200          # below 1 ms per iteration
    assert profiler.reps_for(1_000_000) == 100
    assert profiler.reps_for(4_999_999) == 100        # below 5 ms
    assert profiler.reps_for(5_000_000) == 30
    assert profiler.reps_for(10**9) == 30
    assert profiler.reps_for(10, reps=7) == 7         # an explicit count wins
    # nearest-rank P99 is the maximum only for the 30-sample points
    for n, from_top in ((200, 3), (100, 2), (30, 1)):
        assert n - int(np.ceil(0.99 * n)) + 1 == from_top


def test_report_on_the_cumulative_maximum():
    from paper_2609_07883_b200 import build

    build.build()
    from paper_2609_07883_b200 import profiler

    # the worked example of the monotonisation pin: raw chunk costs {100,140,135,180,260,255,400}
    raw = [100, 140, 135, 180, 260, 255, 400]
    table = {"n_grid": [4], "ctx_grid": [1000], "prefix_grid": [0], "chunk_grid": [16, 32, 48, 64, 80, 96, 112],
             "p99_ns": [[[raw]]], "p50_ns": [[[[x - 1 for x in raw]]]]}
    rep = profiler.monotone_report(table, profiler.to_cost_table(table))
    assert rep["points"] == 7 and rep["raised"] == 2            # 135 -> 140 and 255 -> 260
    assert rep["raised_by_more_than_5_percent"] == 0
    assert rep["max_raise"] == pytest.approx(140 / 135)
    assert rep["mean_raise_of_raised"] == pytest.approx((140 / 135 + 260 / 255) / 2)


def test_clock_record_of_a_window():
    from paper_2609_07883_b200.clocks import ClockSampler

    s = ClockSampler(0)
    s.rows = [(10.00, 1965.0, 1965.0, 300.0, []), (10.05, 1500.0, 1965.0, 990.0, ["sw_power_cap"]),
              (10.10, 1480.0, 1965.0, 1001.0, ["sw_power_cap"]), (10.15, 1520.0, 1965.0, 995.0, ["sw_power_cap"]),
              (10.20, 1965.0, 1965.0, 250.0, [])]
    w = s.window(10.04, 10.16)
    assert w == {"sm_mhz": 1500.0, "sm_max_mhz": 1965.0, "power_w_max": 1001.0, "reasons": ["sw_power_cap"], "samples": 3}
    assert s.window(10.201, 10.202)["samples"] == 1            # shorter than the sampling period: the nearest sample
    s.rows = []
    assert s.window(0, 1)["reasons"] == ["unavailable"]

"""Pins of the oracle's residual table (Sec. 3.3, Sec. 5.1): small cases worked by hand and library routines."""
import numpy as np

from oracle.sw_oracle import ResidualTable


def test_buckets_are_upper_edges_and_overflow_goes_last():
    b = ResidualTable.bucket
    edges = [1, 8, 64]
    assert [b(v, edges) for v in (0, 1, 2, 8, 9, 64, 65, 10**6)] == [0, 0, 1, 1, 2, 2, 2, 2]


def test_nearest_rank_percentile_by_hand_and_against_numpy():
    nr = ResidualTable.nearest_rank
    vals = list(range(1, 101))                       # 1..100: the p-th percentile is p
    assert nr(vals, 990_000) == 99 and nr(vals, 500_000) == 50 and nr(vals, 1_000_000) == 100 and nr(vals, 1) == 1
    assert nr([7], 990_000) == 7
    assert nr([5, 1, 9], 990_000) == 9 and nr([5, 1, 9], 340_000) == 5 and nr([5, 1, 9], 333_333) == 1
    rng = np.random.default_rng(0)
    for _ in range(50):
        v = rng.integers(0, 10**6, size=int(rng.integers(1, 200)))
        p = int(rng.integers(1, 1_000_001))
        # numpy's "inverted_cdf" is the nearest-rank definition
        assert nr(list(v), p) == int(np.percentile(v, p / 1e4, method="inverted_cdf"))


def test_residuals_are_one_sided_windowed_and_per_bucket():
    t = ResidualTable([4, 16], [0, 256, 4096], window=3)
    t.record(2, 100, predicted_ns=1000, observed_ns=900)      # over-prediction counts as zero
    assert t.margin(2, 100) == 0
    for obs in (1100, 1500, 1200):
        t.record(2, 100, 1000, obs)
    # window 3: the zero has been dropped, residuals 100, 500, 200 remain
    assert t.kept[0][1] == [100, 500, 200]
    assert t.margin(2, 100, percentile_ppm=990_000) == 500
    assert t.margin(2, 100, percentile_ppm=500_000) == 200
    # other buckets are untouched: decode-only (c = 0) has no samples and yields the floor
    assert t.margin(2, 0, floor_ns=77) == 77
    assert t.records == 4


def test_margin_is_the_running_maximum_over_smaller_buckets():
    t = ResidualTable([4, 16, 64], [0, 256, 4096], window=8)
    t.record(3, 200, 0, 900)        # bucket (0, 1)
    t.record(10, 3000, 0, 400)      # bucket (1, 2)
    t.record(50, 0, 0, 50)          # bucket (2, 0)
    assert t.margin(3, 200) == 900
    assert t.margin(10, 3000) == 900             # (0,1) lies below (1,2) in both coordinates
    assert t.margin(10, 0) == 0                  # only buckets with c-bucket 0 and n-bucket <= 1: no samples
    assert t.margin(50, 0) == 50
    assert t.margin(50, 4096) == 900
    # nondecreasing in both arguments on a random fill
    rng = np.random.default_rng(1)
    for _ in range(300):
        t.record(int(rng.integers(0, 80)), int(rng.integers(0, 5000)), 1000, int(rng.integers(0, 3000)))
    grid_n, grid_c = [0, 4, 5, 16, 17, 64, 100], [0, 1, 256, 257, 4096, 9000]
    m = np.array([[t.margin(n, c) for c in grid_c] for n in grid_n])
    assert (np.diff(m, axis=0) >= 0).all() and (np.diff(m, axis=1) >= 0).all()


def test_min_samples_floor_and_fallback_signal():
    t = ResidualTable([8], [0, 4096], window=100)
    for k in range(5):
        t.record(4, 512, 1000, 1000 + 10 * k)
    assert t.margin(4, 512, min_samples=6, floor_ns=123) == 123      # too few samples: the floor
    assert t.margin(4, 512, min_samples=5, floor_ns=0) == 40
    assert t.margin(4, 512, min_samples=5, floor_ns=123) == 123      # the empty decode-only bucket below it holds the floor
    assert not t.exceeds(4, 512, configured_margin_ns=40)
    assert t.exceeds(4, 512, configured_margin_ns=39)
    assert not t.exceeds(4, 0, configured_margin_ns=0)                # an empty bucket never signals

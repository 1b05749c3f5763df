"""The iteration-level serving loop on CPU: the controller is the library's (host-only), the executor is the analytic
cost model of Sec. 4.1, so the loop's scheduling semantics and Proposition 1 can be checked without a GPU."""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W

MS = 1_000_000


@pytest.fixture(scope="module")
def env(oracle):
    from paper_2609_07883_b200 import build

    build.build()
    from paper_2609_07883_b200 import binding as B
    from paper_2609_07883_b200 import serving

    n_values = list(range(1, 97))
    chunk_grid = list(range(0, 2049))
    cost = np.array([[oracle.analytic_cost_ns(n, c) for c in chunk_grid] for n in n_values], dtype=np.int64)
    table = B.CostTable(n_values, [1 << 40], [1 << 30], chunk_grid, cost.reshape(len(n_values), 1, 1, -1))

    def execute(batch):
        return oracle.analytic_cost_ns(batch.num_decode, batch.chunk_len)

    trace = W.bursty_trace(num_requests=120, rate_low=20.0, rate_high=80.0, mean_dwell_s=1.0, prompt_median=600.0,
                           prompt_clip=(32, 4096), mean_output=40.0, rng=np.random.default_rng(5))
    return B, serving, table, execute, trace


def test_sloweave_meets_every_deadline_under_an_exact_monotone_cost(env):
    B, serving, table, execute, trace = env
    res = serving.run_trace(trace, 25.0, table, execute, W.LLAMA, 8192, policy="sloweave", c_max=2048, margin_ppm=0,
                            quantum=16, max_decode=96)
    assert res["deadline_misses_with_chunk"] == 0            # Proposition 1 (i)
    assert res["deadline_misses_decode_only"] == res["decode_infeasible_flags"] == 0   # n <= 96 decodes fit 25 ms
    assert res["prefill_tokens"] == int(trace["prompt_len"].sum())
    assert res["requests_meeting_tpot"] == 120
    assert res["tpot_ms_p99_of_request_p99"] <= 25.0
    assert res["chunk_iterations"] > 0 and res["mean_chunk"] > 16


def test_a_large_fixed_chunk_misses_deadlines_that_sloweave_meets(env):
    B, serving, table, execute, trace = env
    fixed = serving.run_trace(trace, 10.0, table, execute, W.LLAMA, 8192, policy="fixed:2048", c_max=2048, max_decode=96)
    adaptive = serving.run_trace(trace, 10.0, table, execute, W.LLAMA, 8192, policy="sloweave", c_max=2048, margin_ppm=0,
                                 max_decode=96)
    assert fixed["deadline_misses_with_chunk"] > 0
    assert adaptive["deadline_misses_with_chunk"] == 0
    assert adaptive["prefill_tokens"] == fixed["prefill_tokens"] == int(trace["prompt_len"].sum())


def test_arrivals_become_eligible_at_iteration_end_and_tokens_add_up(env):
    B, serving, table, execute, trace = env
    seen = []

    def spy(batch):
        seen.append((batch.num_decode, batch.chunk_len, int(batch.total_decode_ctx)))
        return execute(batch)

    res = serving.run_trace(trace, 25.0, table, spy, W.LLAMA, 8192, policy="sloweave", c_max=2048, margin_ppm=0,
                            max_decode=96)
    assert len(seen) == res["iterations"]
    # every iteration decodes one token per active request: decode tokens = sum(output) - one first token per request
    # (the first token comes out of the iteration that finishes the prompt)
    assert sum(n for n, _, _ in seen) == int(trace["output_len"].sum()) - int((trace["output_len"] >= 1).sum())
    assert sum(c for _, c, _ in seen) == int(trace["prompt_len"].sum())
    assert res["ttft_ms_p50"] > 0 and res["trace_duration_s"] * 1e9 >= trace["arrival_ns"][-1]


def test_several_prompts_per_iteration_by_first_fit(env):
    """max_prefills > 1: whole prompts are admitted oldest first while the total fits, the first that does not is cut;
    every token is prefilled exactly once, no admitted list misses a deadline, and fewer iterations carry a chunk."""
    B, serving, table, execute, trace = env
    seen = []

    def spy(batch):
        seen.append(batch)
        return execute(batch)

    one = serving.run_trace(trace, 25.0, table, execute, W.LLAMA, 8192, policy="sloweave", c_max=2048, margin_ppm=0,
                            quantum=16, max_decode=96)
    many = serving.run_trace(trace, 25.0, table, spy, W.LLAMA, 8192, policy="sloweave", c_max=2048, margin_ppm=0,
                             quantum=16, max_decode=96, max_prefills=8)
    assert many["prefill_tokens"] == one["prefill_tokens"] == int(trace["prompt_len"].sum())
    assert many["deadline_misses_with_chunk"] == 0
    assert many["mean_prompts_per_chunk_iteration"] > 1.05
    assert many["chunk_iterations"] < one["chunk_iterations"]
    multi = [b for b in seen if b.chunk_lens is not None]
    assert multi, "no iteration carried more than one prompt"
    for b in multi:
        assert 2 <= len(b.chunk_lens) <= 8 and int(b.chunk_lens.sum()) == b.chunk_len <= 2048
        assert b.chunk_page_indptr[-1] == len(b.prefill_pages)
        order = b.chunk_prefix_lens + b.chunk_lens
        assert (np.diff(order) <= 0).all()               # the longest (prefix + chunk) first
        for P, C, row0, pages in b.chunks():
            assert len(pages) == -(-(P + C) // 16)


def test_heterogeneous_objectives_and_class_margins(env):
    """Per-request objectives D_i (Sec. 3.4): a 10 ms interactive class shares the batch with a 50 ms class.  The budget
    is the minimum over the active requests, so the tight class is protected whenever one of its requests is active and
    the loose one never misses either; a class margin delta_i only tightens the budget."""
    B, serving, table, execute, trace = env
    rng = np.random.default_rng(12)
    tight = rng.random(len(trace["arrival_ns"])) < 0.3
    mixed = dict(trace, tpot_ms=np.where(tight, 10.0, 50.0))
    res = serving.run_trace(mixed, 25.0, table, execute, W.LLAMA, 8192, policy="sloweave", c_max=2048, margin_ppm=0,
                            quantum=16, max_decode=96)
    assert res["deadline_misses_with_chunk"] == 0
    assert res["requests_meeting_tpot"] == len(tight)            # every request meets its OWN objective
    loose_only = serving.run_trace(dict(trace, tpot_ms=np.full(len(tight), 50.0)), 25.0, table, execute, W.LLAMA, 8192,
                                   policy="sloweave", c_max=2048, margin_ppm=0, quantum=16, max_decode=96)
    tight_only = serving.run_trace(dict(trace, tpot_ms=np.full(len(tight), 10.0)), 25.0, table, execute, W.LLAMA, 8192,
                                   policy="sloweave", c_max=2048, margin_ppm=0, quantum=16, max_decode=96)
    # the mixture sits between the two pure cases: slack of the loose class is used when no tight request is active
    assert tight_only["mean_chunk"] <= res["mean_chunk"] <= loose_only["mean_chunk"]
    assert tight_only["mean_chunk"] < loose_only["mean_chunk"]
    # a 2 ms margin for the tight class shrinks the chunks further and still meets everything
    guarded = serving.run_trace(dict(mixed, margin_ms=np.where(tight, 2.0, 0.0)), 25.0, table, execute, W.LLAMA, 8192,
                                policy="sloweave", c_max=2048, margin_ppm=0, quantum=16, max_decode=96)
    assert guarded["deadline_misses_with_chunk"] == 0 and guarded["requests_meeting_tpot"] == len(tight)
    assert guarded["mean_chunk"] <= res["mean_chunk"]
    assert guarded["tpot_ms_p99_of_request_p99"] <= 50.0

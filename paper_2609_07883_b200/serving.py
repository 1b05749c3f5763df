"""Iteration-level serving loop that drives the CUDA path with the SLOWeave controller (the bursty end-to-end workload).

Each iteration decodes one token for every active request and optionally processes one prefill chunk of the oldest
pending request (Sec. 4.1); requests that arrive during an iteration become eligible at its end.  The chunk is chosen
by ``sw_choose_chunk`` (Algorithm 1) from the measured cost table; the iteration itself is one launch per layer (KV append
and mixed attention together) over a stack of ``layers`` KV pools, and the virtual clock advances by its measured device time.
Orchestration and bookkeeping only: chunk choice, append and attention all run in the library.
"""
from __future__ import annotations

import argparse
import json
import sys
import time
from collections import deque
from pathlib import Path

import numpy as np

from . import workloads as W

MS = 1_000_000


class PagePool:
    """Free list of page ids (host side)."""

    def __init__(self, num_pages: int, rng: np.random.Generator):
        self.free = list(rng.permutation(num_pages).astype(np.int32))

    def take(self, k: int):
        if k > len(self.free):
            return None
        out = self.free[-k:] if k else []
        del self.free[len(self.free) - k:]
        return out

    def give(self, ids):
        self.free.extend(ids)


class Request:
    __slots__ = ("rid", "arrival", "prompt", "output", "prefilled", "generated", "pages", "last_token", "first_token",
                 "gaps", "done_at", "D_ns", "margin_ns")

    def __init__(self, rid, arrival, prompt, output, D_ns, margin_ns=0):
        self.rid, self.arrival, self.prompt, self.output = rid, int(arrival), int(prompt), int(output)
        self.D_ns = int(D_ns)            # the request's own token-gap objective D_i (Sec. 3.4, heterogeneous SLOs)
        self.margin_ns = int(margin_ns)  # the prediction margin delta_i reserved for its class
        self.prefilled = 0
        self.generated = 0
        self.pages = None
        self.last_token = 0
        self.first_token = None
        self.gaps = []
        self.done_at = None


def gpu_executor(ctx, pools, shape: W.AttnShape, c_max: int, max_decode: int, seed: int = W.SEED_BASE + 44):
    """Returns execute(batch) -> measured device nanoseconds of one iteration over the layer stack: per layer one
    launch that appends the new K/V rows and runs the mixed attention, timed with CUDA events on the current stream."""
    import torch

    from . import binding as B

    dev = pools[0].device
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    rows_max = c_max + max_decode
    q = torch.randn(rows_max, shape.num_q_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    k_new = torch.randn(rows_max, shape.num_kv_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    v_new = torch.randn(rows_max, shape.num_kv_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    out = torch.empty_like(q)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def execute(batch: W.MixedBatch) -> int:
        db = B.DeviceBatch(batch, dev)
        rows = batch.num_rows
        ev0.record()
        for pool_t in pools:
            B.sw_mixed_iteration_run(ctx, pool_t, db, k_new[:rows], v_new[:rows], q[:rows], out[:rows])
        ev1.record()
        ev1.synchronize()
        return int(ev0.elapsed_time(ev1) * 1e6)

    return execute


def run_trace(trace: dict, tpot_ms: float, table, execute, shape: W.AttnShape, num_pages: int, policy: str = "sloweave",
              c_max: int = 4096, margin_ppm: int = 50_000, margin_abs_ns: int = 0, quantum: int = 16, max_decode: int = 512,
              ctx_cap: int | None = None, seed: int = W.SEED_BASE + 44, log=None, page_tables: bool = True,
              ttft_slo_ms: float | None = None, telemetry=None, fallback_margin_ns: int | None = None,
              residual_percentile_ppm: int = 990_000, residual_min_samples: int = 8, fallback_hold: int = 8,
              max_prefills: int = 1, prefix_cap: int | None = None, reprofile=None,
              reprofile_after_fallbacks: int = 64) -> dict:
    """Run the whole trace; returns statistics.  ``policy`` is "sloweave" or "fixed:<chunk>".  ``execute(batch)`` runs
    one iteration and returns its duration in ns (``gpu_executor`` for the CUDA path).  ``ctx_cap`` clamps the total
    context passed to the table lookup to the table's last grid point.  ``page_tables=False`` hands ``execute`` a batch
    without page lists (enough for a cost model that looks only at sizes; the simulator study runs that way).  With
    ``ttft_slo_ms`` the result also counts the requests that meet both SLOs and the goodput (Sec. 4.3).

    ``telemetry`` (a ``binding.Telemetry``) closes the feedback loop of Sec. 3.3 / Sec. 5.1: every iteration's raw table
    prediction and measured duration are recorded, the residual table's margin for (n, L) is added to the controller's
    margin, and, when ``fallback_margin_ns`` is given and the residuals exceed it, the iteration runs decode-only.  So
    that a stale residual cannot starve the queue, at most ``fallback_hold`` consecutive iterations fall back; the next
    one admits a chunk again under the residual margin and so refreshes the residuals.

    ``reprofile`` (a callable returning a fresh ``binding.CostTable``) is the re-profiling hook of Sec. 5.1: after
    ``reprofile_after_fallbacks`` fallback iterations since the last table the loop asks for a new table and starts a
    new residual window (the telemetry object's old residuals age out of its sliding window).

    ``max_prefills > 1`` (SLOWeave policy only) admits several pending prompts per iteration by first fit
    (``sw_choose_chunks``, Sec. 3.3 "Prefill batching"): whole prompts oldest first while the prediction for the total
    still meets the budget, the first one that does not fit cut by the bisection; the iteration then carries one
    prefill chunk per admitted prompt.  ``prefix_cap`` (the table's last prefix grid point) bounds the summed prefix
    lengths of the candidates, which is the prefix coordinate the first-fit prediction is looked up at."""
    from . import binding as B

    S = shape.page_size
    D_ns = int(tpot_ms * MS)
    rng = np.random.default_rng(seed)
    pool = PagePool(num_pages, rng)
    # per-request objectives D_i and class margins delta_i (optional trace columns "tpot_ms" / "margin_ms")
    tpot_of = trace.get("tpot_ms")
    margin_of = trace.get("margin_ms")
    reqs = [Request(i, trace["arrival_ns"][i], trace["prompt_len"][i], trace["output_len"][i],
                    (float(tpot_of[i]) if tpot_of is not None else tpot_ms) * MS,
                    (float(margin_of[i]) if margin_of is not None else 0.0) * MS)
            for i in range(len(trace["arrival_ns"]))]
    fixed_chunk = int(policy.split(":")[1]) if policy.startswith("fixed:") else None

    pending, active = deque(), []
    nxt, now, done = 0, 0, 0
    iters = chunk_iters = 0
    misses_chunk = misses_decode_only = infeasible_flags = stalled_for_memory = 0
    chunks, iter_ns, pred_err, pred_ratio = [], [], [], []
    fallback_iters = fallback_run = 0
    fallbacks_since_table = reprofiles = 0
    prompts_per_chunk_iter = []
    miss_samples = []        # the first few iterations that ran a chunk and overran the earliest deadline
    prefill_tokens = 0
    wall0 = time.time()
    while done < len(reqs):
        while nxt < len(reqs) and reqs[nxt].arrival <= now:
            pending.append(reqs[nxt])
            nxt += 1
        if not pending and not active:
            now = reqs[nxt].arrival
            continue
        # ---- the controller's decision -----------------------------------------------------------------------
        head = pending[0] if pending else None
        if head is not None and head.pages is None:
            need = -(-(head.prompt + head.output) // S)
            head.pages = pool.take(need)           # blocks for the whole request are reserved when it is first scheduled
            if head.pages is None:
                stalled_for_memory += 1
                head = None
        n = len(active)
        if n >= max_decode and head is not None:
            head = None                             # the decode batch is full: no new request can finish its prefill
        remaining = head.prompt - head.prefilled if head is not None else 0
        # d_i = l_i + D_i, less the margin delta_i reserved for the request's class: B = min_i(d_i - delta_i) - now
        deadlines = np.array([r.last_token + r.D_ns - r.margin_ns for r in active], dtype=np.int64)
        true_deadline = min((r.last_token + r.D_ns for r in active), default=0)
        total_ctx = sum(r.prompt + r.generated for r in active)
        if ctx_cap is not None:
            total_ctx = min(total_ctx, ctx_cap)
        budget = int(deadlines.min() - now) if n else 0
        predicted = 0
        flags = 0
        admitted = None      # [(request, tokens)] when several prompts share the iteration
        fell_back = False
        extra_margin = 0
        if telemetry is not None and fixed_chunk is None and n and remaining:
            L_now = min(c_max, remaining)
            extra_margin = telemetry.margin(n, L_now, residual_percentile_ppm, residual_min_samples, 0)
            if fallback_margin_ns is not None and fallback_run < fallback_hold and \
                    telemetry.exceeds(n, L_now, fallback_margin_ns, residual_percentile_ppm, residual_min_samples):
                fell_back = True
        if fell_back:
            c = 0
            fallback_run += 1
            fallback_iters += 1
            fallbacks_since_table += 1
            if reprofile is not None and fallbacks_since_table >= reprofile_after_fallbacks:
                table = reprofile()
                telemetry.reset()          # residuals against the old table say nothing about the new one
                reprofiles += 1
                fallbacks_since_table = 0
        elif fixed_chunk is not None:
            c = min(fixed_chunk, remaining)
        elif max_prefills > 1 and head is not None:
            # first fit over the oldest pending requests (each needs its blocks reserved before it can be scheduled)
            cands, prefix_total = [], 0
            for r in list(pending)[:min(max_prefills, B.SW_MAX_CHUNKS, max(1, max_decode - n))]:
                if cands and prefix_cap is not None and prefix_total + r.prefilled > prefix_cap:
                    break
                prefix_total += r.prefilled
                if r.pages is None:
                    r.pages = pool.take(-(-(r.prompt + r.output) // S))
                    if r.pages is None:
                        break
                cands.append(r)
            fallback_run = 0
            lens_adm, ch = B.sw_choose_chunks(table if n else None, now, deadlines, total_ctx, [r.prefilled for r in cands],
                                              [r.prompt - r.prefilled for r in cands], c_max=c_max, chunk_quantum=1,
                                              margin_abs_ns=margin_abs_ns + extra_margin, margin_ppm=margin_ppm)
            admitted = list(zip(cands, lens_adm))
            c, flags, predicted = ch.chunk, ch.flags, ch.predicted_ns
        else:
            q_eff = quantum if remaining >= quantum else 1   # the last few tokens of a prompt are below the quantum
            prefilled = head.prefilled if head else 0
            fallback_run = 0
            m_abs = margin_abs_ns + extra_margin
            ch = B.sw_choose_chunk(table if n else None, now, deadlines, total_ctx, prefilled, remaining,
                                   c_max=c_max, chunk_quantum=q_eff, margin_abs_ns=m_abs, margin_ppm=margin_ppm)
            L = min(c_max, remaining)
            if q_eff > 1 and L % q_eff and ch.chunk == L - L % q_eff:
                # The quantum stopped just short of L.  If L itself fits the budget, take it: a prompt's last few tokens
                # would otherwise cost a whole extra iteration.
                fine = B.sw_choose_chunk(table if n else None, now, deadlines, total_ctx, prefilled, remaining, c_max=c_max,
                                         chunk_quantum=1, margin_abs_ns=m_abs, margin_ppm=margin_ppm)
                if fine.chunk == L:
                    ch = fine
            c, flags, predicted = ch.chunk, ch.flags, ch.predicted_ns
        if n == 0 and c == 0:
            # nothing to run (memory stall with an idle GPU): wait for the next arrival or fail loudly
            if nxt < len(reqs):
                now = max(now, reqs[nxt].arrival)
                continue
            raise RuntimeError("serving loop stalled: pool too small for the remaining requests")
        # ---- build the iteration and run it over the layer stack -----------------------------------------------
        if admitted is None:
            admitted = [(head, c)] if c > 0 else []
        P = admitted[0][0].prefilled if admitted else 0
        lens = np.array([r.prompt + r.generated for r in active], dtype=np.int32)
        per = [(-(-int(L) // S)) for L in lens]
        indptr = np.zeros(n + 1, dtype=np.int32)
        indptr[1:] = np.cumsum(per)
        if page_tables:
            dpages = np.concatenate([np.asarray(r.pages[:k], dtype=np.int32) for r, k in zip(active, per)]) if n else \
                np.zeros(0, np.int32)
            ppages = np.asarray(head.pages[: -(-(P + c) // S)], dtype=np.int32) if c > 0 else np.zeros(0, np.int32)
        else:
            dpages = ppages = np.zeros(0, np.int32)
        if len(admitted) > 1:
            # one chunk per admitted prompt, the longest (prefix + chunk) first: that is the order they are scheduled in
            order = sorted(admitted, key=lambda rc: -(rc[0].prefilled + rc[1]))
            lists = [np.asarray(r.pages[: -(-(r.prefilled + cj) // S)], dtype=np.int32) if page_tables else
                     np.zeros(0, np.int32) for r, cj in order]
            cp_indptr = np.zeros(len(order) + 1, dtype=np.int32)
            cp_indptr[1:] = np.cumsum([len(x) for x in lists])
            batch = W.MixedBatch(shape, num_pages, order[0][0].prefilled, c, np.concatenate(lists), lens, indptr, dpages,
                                 chunk_prefix_lens=np.array([r.prefilled for r, _ in order], dtype=np.int32),
                                 chunk_lens=np.array([cj for _, cj in order], dtype=np.int32), chunk_page_indptr=cp_indptr)
        else:
            batch = W.MixedBatch(shape, num_pages, P, c, ppages, lens, indptr, dpages)
        dt = int(execute(batch))
        now += dt
        iters += 1
        iter_ns.append(dt)
        # ---- bookkeeping ------------------------------------------------------------------------------------------
        if n and now > true_deadline:
            if c > 0:
                misses_chunk += 1
                if len(miss_samples) < 16:
                    miss_samples.append({"n": n, "total_ctx": int(total_ctx), "chunks": [int(cj) for _, cj in admitted],
                                         "prefixes": [int(r.prefilled) for r, _ in admitted], "budget_ns": budget,
                                         "predicted_ns": int(predicted), "measured_ns": dt,
                                         "late_ns": int(now - true_deadline)})
            else:
                misses_decode_only += 1
        if flags & B.SW_F_DECODE_INFEASIBLE:
            infeasible_flags += 1
        if predicted and n:
            pred_err.append(dt - predicted)
            pred_ratio.append(predicted / max(dt, 1))
        if telemetry is not None and n:
            # the table's own prediction, without any margin (several chunks: total tokens at the summed prefix)
            raw = table.lookup(n, total_ctx, sum(r.prefilled for r, _ in admitted) if admitted else 0, c)
            telemetry.record(n, c, raw, dt, slack_ns=budget - dt, fallback=fell_back)
        still = []
        for r in active:
            r.generated += 1
            r.gaps.append(now - r.last_token)
            r.last_token = now
            if r.generated >= r.output:
                r.done_at = now
                pool.give(r.pages)
                r.pages = None
                done += 1
            else:
                still.append(r)
        active = still
        if c > 0:
            chunk_iters += 1
            chunks.append(c)
            prefill_tokens += c
            prompts_per_chunk_iter.append(len(admitted))
        for head, cj in admitted:                  # admitted prompts are the oldest pending ones, in queue order
            head.prefilled += cj
            if head.prefilled >= head.prompt:      # the iteration that finishes the prompt emits the first token
                assert pending[0] is head
                pending.popleft()
                head.first_token = now
                head.last_token = now
                head.generated = 1
                if head.output <= 1:
                    head.done_at = now
                    pool.give(head.pages)
                    head.pages = None
                    done += 1
                else:
                    active.append(head)
        if log and iters % 2000 == 0:
            log(f"  iter {iters}: t={now / 1e9:.2f}s done={done} active={len(active)} pending={len(pending)} "
                f"wall={time.time() - wall0:.0f}s")
    ttft = np.array([r.first_token - r.arrival for r in reqs], dtype=np.float64) / MS
    p99_gap = np.array([np.percentile(r.gaps, 99) if r.gaps else 0.0 for r in reqs]) / MS
    duration_s = now / 1e9
    tpot_each = np.array([r.D_ns for r in reqs], dtype=np.float64) / MS
    slo = {}
    if ttft_slo_ms is not None:
        both = int(np.sum((ttft <= ttft_slo_ms) & (p99_gap <= tpot_each)))
        slo = {"ttft_slo_ms": ttft_slo_ms, "requests_meeting_both_slos": both, "slo_attainment": both / len(reqs),
               "goodput_rps": both / duration_s, "throughput_rps": len(reqs) / duration_s}
    return {
        **slo,
        "policy": policy, "tpot_ms": tpot_ms, "requests": len(reqs), "iterations": iters, "chunk_iterations": chunk_iters,
        "deadline_misses_with_chunk": misses_chunk, "deadline_misses_decode_only": misses_decode_only,
        "decode_infeasible_flags": infeasible_flags, "memory_stalls": stalled_for_memory,
        "trace_duration_s": duration_s, "prefill_tokens": prefill_tokens,
        "prefill_tokens_per_s": prefill_tokens / duration_s, "decode_tokens_per_s": float(sum(r.output for r in reqs)) / duration_s,
        "mean_chunk": float(np.mean(chunks)) if chunks else 0.0, "p99_chunk": float(np.percentile(chunks, 99)) if chunks else 0.0,
        "iter_ms_p50": float(np.percentile(iter_ns, 50)) / MS, "iter_ms_p99": float(np.percentile(iter_ns, 99)) / MS,
        "ttft_ms_p50": float(np.percentile(ttft, 50)), "ttft_ms_p99": float(np.percentile(ttft, 99)),
        "tpot_ms_p99_of_request_p99": float(np.percentile(p99_gap, 99)),
        "requests_meeting_tpot": int(np.sum(p99_gap <= tpot_each)),
        "prediction_error_ms_p99": float(np.percentile(pred_err, 99)) / MS if pred_err else 0.0,
        "predicted_over_measured_mean": float(np.mean(pred_ratio)) if pred_ratio else 0.0,
        "predicted_over_measured_p50": float(np.median(pred_ratio)) if pred_ratio else 0.0,
        "fallback_iterations": fallback_iters, "reprofiles": reprofiles,
        "mean_prompts_per_chunk_iteration": float(np.mean(prompts_per_chunk_iter)) if prompts_per_chunk_iter else 0.0,
        "margin_ppm": margin_ppm, "c_max": c_max, "quantum": quantum, "wall_s": time.time() - wall0,
        "miss_samples": miss_samples,
    }


def main(argv=None):
    import torch

    from . import binding as B
    from . import build, profiler

    ap = argparse.ArgumentParser(description="bursty serving loop over a layer stack with the SLOWeave controller")
    ap.add_argument("--requests", type=int, default=2000)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--pages", type=int, default=40960, help="pages per layer pool")
    ap.add_argument("--tpot-ms", type=float, nargs="+", default=[10.0, 25.0])
    ap.add_argument("--policies", nargs="+", default=["sloweave"])
    ap.add_argument("--rate-scale", type=float, nargs="+", default=[1.0],
                    help="divide the trace's arrival times by this factor (1 = the stated 2 / 20 req/s)")
    ap.add_argument("--c-max", type=int, default=4096)
    ap.add_argument("--margin-ppm", type=int, default=50_000)
    ap.add_argument("--table", default=None, help="JSON cost table to reuse; measured first when absent")
    ap.add_argument("--table-reps", type=int, default=0,
                    help="timed iterations per grid point; 0 = by the point's duration (200 below 1 ms, 100 below 5 ms, else 30)")
    ap.add_argument("--max-prefills", type=int, default=1, help="prompts admitted per iteration (first fit when > 1)")
    ap.add_argument("--ttft-slo-ms", type=float, default=None,
                    help="also count the requests that meet both SLOs and the goodput (Sec. 4.3)")
    ap.add_argument("--telemetry", action="store_true",
                    help="residual feedback (Sec. 3.3): add the P99 residual of the (n, L) bin to the controller's margin")
    ap.add_argument("--out", default="bursty_results.json")
    args = ap.parse_args(argv)

    build.build()
    dev = torch.device("cuda", 0)
    shape = W.LLAMA
    max_decode = 512
    ctx = B.Context(shape, args.pages, args.c_max, max_decode, args.pages + 64)
    pools = []
    for layer in range(args.layers):
        t = torch.empty(args.pages * shape.page_elems, dtype=torch.bfloat16, device=dev)
        W.fill_normal_bf16_(t, W.SEED_BASE + 400 + layer)
        pools.append(t)
    log = lambda s: print(s, file=sys.stderr, flush=True)
    if args.table and Path(args.table).exists():
        tab = profiler.load_table(args.table)
    else:
        tokens = args.pages * shape.page_size
        n_grid = [1, 4, 16, 48, 128, 256, 512]
        prefix_grid = [0, 2048, 8192, 32768]
        chunk_grid = [0, 16, 64, 128, 256, 512, 1024, 2048, 4096]
        # the largest context that still leaves room for the longest prompt piece and one ragged page per request
        ctx_top = tokens - (prefix_grid[-1] + chunk_grid[-1]) - shape.page_size * (n_grid[-1] + 64)
        ctx_grid = [t for t in (8192, 16384, 32768, 65536, 131072, 196608, 393216) if t < ctx_top] + [ctx_top]
        log(f"measuring cost table: {len(n_grid) * len(ctx_grid) * len(prefix_grid) * len(chunk_grid)} points, {args.layers} layers")
        tab = profiler.measure_table(ctx, pools, shape, args.pages, n_grid, ctx_grid, prefix_grid, chunk_grid,
                                     reps=args.table_reps, warmup=3, progress=log, fused=True)
        if args.table:
            profiler.save_table(tab, args.table)
    table = profiler.to_cost_table(tab)
    stats = profiler.monotone_report(tab, table)
    log("cost table: " + json.dumps(stats))
    trace = W.bursty_trace(num_requests=args.requests)
    execute = gpu_executor(ctx, pools, shape, args.c_max, max_decode)
    results = {"layers": args.layers, "pages_per_layer": args.pages, "table_points": int(np.prod(np.shape(tab["p99_ns"]))),
               "table_stats": stats, "runs": []}
    for scale in args.rate_scale:
        scaled = dict(trace, arrival_ns=(trace["arrival_ns"] / scale).astype(np.int64))
        for tpot in args.tpot_ms:
            for policy in args.policies:
                log(f"run: rate x{scale} tpot={tpot} ms policy={policy}")
                tele = B.Telemetry([1, 4, 16, 48, 128, 256], [0, 64, 256, 1024, 2048, 4096]) if args.telemetry else None
                res = run_trace(scaled, tpot, table, execute, shape, args.pages, policy=policy, c_max=args.c_max,
                                margin_ppm=args.margin_ppm, max_decode=max_decode, ctx_cap=tab["ctx_grid"][-1], log=log,
                                max_prefills=args.max_prefills if policy == "sloweave" else 1, prefix_cap=tab["prefix_grid"][-1],
                                telemetry=tele, ttft_slo_ms=args.ttft_slo_ms)
                B.sw_check_status(ctx)
                if tele is not None:
                    res["telemetry"] = tele.totals()
                    tele.close()
                res["rate_scale"] = scale
                log(json.dumps(res))
                results["runs"].append(res)
    Path(args.out).parent.mkdir(parents=True, exist_ok=True)
    Path(args.out).write_text(json.dumps(results, indent=1))
    print(json.dumps(results))


if __name__ == "__main__":
    main()

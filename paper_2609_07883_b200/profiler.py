"""Start-up profiler: measure the iteration cost T(n, ctx, prefix, c) on a grid with ``sw_cost_probe`` and build the
monotone P99 lookup table the controller searches (Sec. 5.1; Sec. 6.4).

Orchestration only: the timing is done by ``sw_cost_probe`` (CUDA events inside the library), the monotonisation and
the lookups by ``sw_cost_table_create`` / ``sw_cost_table_lookup``.  One grid point = one synthetic iteration with
``n`` decodes of equal context ``ctx / n`` plus a chunk of ``c`` tokens at prefix ``prefix``, run over a stack of
``layers`` KV pools (the chunk axis includes c = 0, the decode-only plane).
"""
from __future__ import annotations

import json
import time
from pathlib import Path

import numpy as np

from . import workloads as W


def probe_batch(shape: W.AttnShape, num_pages: int, n: int, ctx_total: int, prefix: int, chunk: int,
                rng: np.random.Generator) -> W.MixedBatch:
    """A synthetic iteration at one grid point: n decodes sharing ctx_total tokens as evenly as possible."""
    if n > 0:
        base, extra = divmod(max(ctx_total, n), n)
        lens = [base + (1 if i < extra else 0) for i in range(n)]
    else:
        lens = []
    return W.make_batch(shape, num_pages, lens, prefix if chunk > 0 else 0, chunk, rng,
                        name=f"probe_n{n}_ctx{ctx_total}_P{prefix}_C{chunk}")


def pages_needed(shape: W.AttnShape, n: int, ctx_total: int, prefix: int, chunk: int) -> int:
    S = shape.page_size
    per = -(-max(ctx_total, n) // max(n, 1)) if n > 0 else 0
    return n * (-(-per // S) + 1) + -(-(prefix + chunk) // S) + 8


def reps_for(iteration_ns: int, reps: int = 0) -> int:
    """Timed iterations per grid point: at least 200 below 1 ms per iteration, 100 below 5 ms, 30 otherwise, so that the
    nearest-rank 99th percentile (the ceil(0.99 * reps)-th smallest sample) leaves out the two / the one largest sample of
    a short point and is the maximum only for the long ones, where a scheduling hiccup is small beside the iteration.
    ``reps`` > 0 fixes the number instead."""
    if reps > 0:
        return reps
    return 200 if iteration_ns < 1_000_000 else (100 if iteration_ns < 5_000_000 else 30)


def measure_table(ctx, pools, shape: W.AttnShape, num_pages: int, n_grid, ctx_grid, prefix_grid, chunk_grid,
                  reps: int = 0, warmup: int = 3, seed: int = W.SEED_BASE + 40, progress=None, fused: bool = False) -> dict:
    """Probe every grid point (``fused``: with the KV append in every launch, as ``sw_mixed_iteration_run`` runs it).  ``ctx``
    is a binding.Context big enough for the largest point; ``pools`` the layer stack (list of device tensors).  Every point
    gets ``warmup`` untimed iterations (which also size its sample, see ``reps_for``) and then its timed ones.  Returns a
    plain dict (JSON-serialisable) with the median, the nearest-rank 99th percentile, the maximum and the number of timed
    iterations of every point."""
    import torch

    from . import binding as B

    dev = pools[0].device
    rng = np.random.default_rng(seed)
    max_rows = max(chunk_grid) + max(n_grid)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    q = torch.randn(max_rows, shape.num_q_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    out = torch.empty_like(q)
    k_new = v_new = None
    if fused:
        k_new = torch.randn(max_rows, shape.num_kv_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
        v_new = torch.randn(max_rows, shape.num_kv_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    shape4 = (len(n_grid), len(ctx_grid), len(prefix_grid), len(chunk_grid))
    p50 = np.zeros(shape4, dtype=np.int64)
    p99 = np.zeros(shape4, dtype=np.int64)
    top = np.zeros(shape4, dtype=np.int64)
    count = np.zeros(shape4, dtype=np.int64)
    probe = (lambda db, w, r: B.sw_cost_probe_iteration(ctx, pools, db, k_new, v_new, q, out, warmup=w, reps=r)) if fused else (
        lambda db, w, r: B.sw_cost_probe(ctx, pools, db, q, out, warmup=w, reps=r))
    t0 = time.time()
    for a, n in enumerate(n_grid):
        for b, ctx_total in enumerate(ctx_grid):
            for c_i, prefix in enumerate(prefix_grid):
                for e, chunk in enumerate(chunk_grid):
                    if n == 0 and chunk == 0:
                        continue
                    if chunk == 0 and c_i > 0:      # the decode-only plane does not depend on the prefix
                        for plane in (p50, p99, top, count):
                            plane[a, b, c_i, e] = plane[a, b, 0, e]
                        continue
                    batch = probe_batch(shape, num_pages, int(n), int(ctx_total), int(prefix), int(chunk), rng)
                    db = B.DeviceBatch(batch, dev)
                    first, _, _ = probe(db, warmup, 3)          # a look at the point's duration sizes its sample
                    r = reps_for(first, reps)
                    m, h, samples = probe(db, 0, r)
                    p50[a, b, c_i, e], p99[a, b, c_i, e], top[a, b, c_i, e], count[a, b, c_i, e] = m, h, int(samples.max()), r
        if progress:
            progress(f"n={n}: {time.time() - t0:.1f}s")
    B.sw_check_status(ctx)
    return {"n_grid": [int(x) for x in n_grid], "ctx_grid": [int(x) for x in ctx_grid],
            "prefix_grid": [int(x) for x in prefix_grid], "chunk_grid": [int(x) for x in chunk_grid],
            "layers": len(pools), "reps": count.tolist(), "warmup": warmup + 3, "fused_append": bool(fused), "p50_ns": p50.tolist(),
            "p99_ns": p99.tolist(), "max_ns": top.tolist(),
            "percentile_rule": "nearest rank: the ceil(0.99 * reps)-th smallest sample (the maximum when reps < 100)",
            "shape": [shape.num_q_heads, shape.num_kv_heads, shape.head_dim, shape.page_size]}


def save_table(table: dict, path) -> None:
    Path(path).write_text(json.dumps(table))


def load_table(path) -> dict:
    return json.loads(Path(path).read_text())


def to_cost_table(table: dict, interp: bool = False, which: str = "p99_ns"):
    """The controller's table: P99 plane, made monotone by the library (cumulative maximum along every axis)."""
    from . import binding as B

    return B.CostTable(table["n_grid"], table["ctx_grid"], table["prefix_grid"], table["chunk_grid"],
                       np.asarray(table[which], dtype=np.int64), make_monotone=True, interp=interp)


def monotone_report(table: dict, cost_table, which: str = "p99_ns") -> dict:
    """What the library's cumulative maximum did to a measured table: how many grid points it raised, and by how much
    (the raised value over the measured one), read back from the controller's table at every grid point."""
    raw = np.asarray(table[which], dtype=np.float64)
    mono = np.zeros_like(raw)
    for a, n in enumerate(table["n_grid"]):
        for b, c in enumerate(table["ctx_grid"]):
            for d, pre in enumerate(table["prefix_grid"]):
                for e, k in enumerate(table["chunk_grid"]):
                    mono[a, b, d, e] = cost_table.lookup(int(n), int(c), int(pre), int(k))
    live = raw > 0
    ratio = mono[live] / raw[live]
    raised = ratio > 1.0
    p50 = np.asarray(table["p50_ns"], dtype=np.float64)
    spread = raw[live] / np.maximum(p50[live], 1.0)
    return {"points": int(live.sum()), "raised": int(raised.sum()), "raised_by_more_than_5_percent": int((ratio > 1.05).sum()),
            "raised_by_more_than_20_percent": int((ratio > 1.2).sum()),
            "mean_raise_of_raised": float(ratio[raised].mean()) if raised.any() else 1.0, "max_raise": float(ratio.max()),
            "p99_over_p50_mean": float(spread.mean()), "p99_over_p50_max": float(spread.max())}


# --------------------------------------------------------------------------------------------------------------------
# cost-surface sweeps of the named workloads (command line)
# --------------------------------------------------------------------------------------------------------------------
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0


def _work(batch: W.MixedBatch) -> dict:
    sh = batch.shape
    P, C, n, ctx = batch.prefix_len, batch.chunk_len, batch.num_decode, batch.total_decode_ctx
    qo_row = sh.num_q_heads * sh.head_dim * 2 * 2
    return {"decode_bytes": ctx * sh.token_bytes + n * qo_row,
            "prefill_bytes": ((P + C) * sh.token_bytes if C else 0) + C * qo_row,
            "prefill_flops": 4 * sh.num_q_heads * sh.head_dim * (C * P + C * (C + 1) // 2)}


def _timed(ctx, pools, db, q, out, reps: int):
    """(median, P99) nanoseconds per ITERATION over the layer stack; ``reps`` = 0 sizes the sample by the iteration's length."""
    from . import binding as B

    first, _, _ = B.sw_cost_probe(ctx, pools, db, q, out, warmup=3, reps=3)
    p50, p99, _ = B.sw_cost_probe(ctx, pools, db, q, out, warmup=0, reps=reps_for(first, reps))
    return p50, p99


def _with_clocks(rows, spans, sampler):
    """Attach to every row the clock record of the time window in which it was measured."""
    sampler.stop()
    for row, (t0, t1) in zip(rows, spans):
        row["clocks"] = sampler.window(t0, t1)
    return rows


def sweep(config: str, reps: int, log) -> list:
    """Mixed, prefill-only and decode-only launch times over the workload's (prefix, chunk) grid."""
    import json as _json

    import torch

    from . import binding as B
    from .clocks import ClockSampler

    sampler = ClockSampler(0)
    sampler.start()
    spans = []

    peaks_file = Path(__file__).resolve().parent.parent / "MEASURED_PEAKS.json"
    peaks = _json.loads(peaks_file.read_text()) if peaks_file.exists() else {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
    dev = torch.device("cuda", 0)
    shape = W.LLAMA
    if config == "chat":
        grid = [(512, c, n) for n in (16, 64) for c in (64, 128, 256, 512)]
        make = lambda P, C, n: W.chat_batch(n=n, chunk_len=C, prefix_len=P, rng=W.rng_for(1))
        layers, pool_pages = 8, None
    elif config == "mixed":
        grid = [(P, c, 128) for P in (0, 4096, 16384, 28672) for c in (64, 128, 256, 512, 1024, 2048, 4096)]
        make = lambda P, C, n: W.mixed_batch(C, P, n=n, rng=W.rng_for(2))
        layers, pool_pages = 2, None
    else:
        grid = [(98304, c, 16) for c in (1024, 4096, 8192)]
        free, _ = torch.cuda.mem_get_info()
        pool_pages = int(min(120e9, 0.9 * free) // (shape.page_elems * 2))   # ~120 GB pool, live pages scattered over it
        make = lambda P, C, n: W.long_batch(C, P, n=n, num_pages=pool_pages, rng=W.rng_for(3))
        layers = 1
    rows = []
    pools, pool_size = [], 0
    for (P, C, n) in grid:
        batch = make(P, C, n)
        if batch.num_pages != pool_size:
            pools, pool_size = [], batch.num_pages
            torch.cuda.empty_cache()
            for layer in range(layers):
                t = torch.empty(batch.num_pages * shape.page_elems, dtype=torch.bfloat16, device=dev)
                W.fill_normal_bf16_(t, W.SEED_BASE + 500 + layer)
                pools.append(t)
        total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
        ctx = B.Context(shape, batch.num_pages, max(C, 1), max(n, 1), total_pages + 16)
        q = torch.randn(batch.num_rows, shape.num_q_heads, shape.head_dim, device=dev).to(torch.bfloat16)
        out = torch.empty_like(q)
        variants = {"mixed": batch,
                    "prefill_only": W.MixedBatch(shape, batch.num_pages, P, C, batch.prefill_pages, np.zeros(0, np.int32),
                                                 np.zeros(1, np.int32), np.zeros(0, np.int32)),
                    "decode_only": W.MixedBatch(shape, batch.num_pages, 0, 0, np.zeros(0, np.int32), batch.decode_kv_len,
                                                batch.decode_page_indptr, batch.decode_pages)}
        row = {"prefix": P, "chunk": C, "decodes": n, "decode_ctx": batch.total_decode_ctx, "pool_pages": batch.num_pages}
        w = _work(batch)
        t_begin = time.time()
        for name, b in variants.items():
            db = B.DeviceBatch(b, dev)
            qq = q if name != "decode_only" else q[C:]
            p50, p99 = _timed(ctx, pools, db, qq, out[: b.num_rows], reps)
            row[name + "_us_p50"] = p50 / 1e3 / layers
            row[name + "_us_p99"] = p99 / 1e3 / layers
        B.sw_check_status(ctx)
        spans.append((t_begin, time.time()))
        t_pf, t_dec, t_mix = (row[k + "_us_p50"] * 1e-6 for k in ("prefill_only", "decode_only", "mixed"))
        row["prefill_tflops"] = w["prefill_flops"] / t_pf / 1e12
        row["prefill_frac_measured"] = row["prefill_tflops"] / peaks["bf16_tflops"]
        row["prefill_frac_nominal"] = row["prefill_tflops"] / NOMINAL_BF16_TFLOPS
        row["decode_gbs"] = w["decode_bytes"] / t_dec / 1e9
        row["decode_frac_measured"] = row["decode_gbs"] / peaks["hbm_gbs"]
        row["decode_frac_nominal"] = row["decode_gbs"] / NOMINAL_HBM_GBS
        row["prefill_tokens_per_s"] = C / t_mix
        row["decode_tokens_per_s"] = n / t_mix
        row["mixed_vs_sum"] = t_mix / (t_pf + t_dec)
        rows.append(row)
        log(f"P={P:6d} C={C:5d} n={n:4d}  mixed {row['mixed_us_p50']:9.1f} us  prefill {row['prefill_only_us_p50']:9.1f} us "
            f"({row['prefill_tflops']:7.1f} TFLOP/s, {row['prefill_frac_measured']:.2f} of measured, "
            f"{row['prefill_frac_nominal']:.2f} of nominal)  decode {row['decode_only_us_p50']:8.1f} us ({row['decode_gbs']:6.0f} GB/s, "
            f"{row['decode_frac_measured']:.2f} / {row['decode_frac_nominal']:.2f})  mixed/(pf+dec) {row['mixed_vs_sum']:.2f}")
        del ctx
    return _with_clocks(rows, spans, sampler)


def sweep_multichunk(reps: int, log) -> list:
    """One iteration's prefill tokens given as 1, 2, 4 or 8 chunks of different prompts (each at its own prefix), with
    and without the chat workload's 64 decodes: launch times of ``sw_mixed_attn_run``."""
    import torch

    from . import binding as B
    from .clocks import ClockSampler

    sampler = ClockSampler(0)
    sampler.start()
    spans = []
    dev = torch.device("cuda", 0)
    shape = W.LLAMA
    rows = []
    equal = [[(prefix, total // k)] * k for total, prefix in ((512, 512), (2048, 4096)) for k in (1, 2, 4, 8)]
    # chunks of very different lengths: the end of a long prompt beside the start of new ones, and the same tokens as
    # one chunk of the long prompt for comparison
    unequal = [[(28672, 512)], [(28672, 256), (0, 256)], [(28672, 128), (4096, 128), (0, 256)]]
    for chunks in equal + unequal:
        for n in (0, 64):
            rng = W.rng_for(1)
            lens = rng.integers(256, 2048, size=n, endpoint=True) if n else []
            k, total, prefix = len(chunks), sum(c for _, c in chunks), chunks[0][0]
            need = sum(-(-int(x) // 16) for x in lens) + sum(-(-(P + C) // 16) for P, C in chunks) + 64
            batch = W.make_multi_batch(shape, need, lens, chunks, rng)
            pools = []
            for layer in range(4):
                t = torch.empty(batch.num_pages * shape.page_elems, dtype=torch.bfloat16, device=dev)
                W.fill_normal_bf16_(t, W.SEED_BASE + 700 + layer)
                pools.append(t)
            pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
            ctx = B.Context(shape, batch.num_pages, batch.chunk_len, max(n, 1), pages + 16)
            q = torch.randn(batch.num_rows, shape.num_q_heads, shape.head_dim, device=dev).to(torch.bfloat16)
            out = torch.empty_like(q)
            t_begin = time.time()
            p50, p99 = _timed(ctx, pools, B.DeviceBatch(batch, dev), q, out, reps)
            B.sw_check_status(ctx)
            spans.append((t_begin, time.time()))
            flops = 4 * shape.num_q_heads * shape.head_dim * sum(C * P + C * (C + 1) // 2 for P, C in chunks)
            row = {"prefill_tokens": total, "prefix_of_each": prefix, "chunks": k, "decodes": n, "us_p50": p50 / 4e3,
                   "chunk_list": [list(c) for c in chunks],
                   "us_p99": p99 / 4e3, "prefill_gflop": flops / 1e9}
            rows.append(row)
            log(f"tokens {total:5d} in {k} chunk(s) {chunks if len(set(chunks)) > 1 else 'at prefix ' + str(prefix)}, {n:3d} decodes: {row['us_p50']:8.1f} us "
                f"(p99 {row['us_p99']:.1f}), {flops / 1e9:.1f} GFLOP of prefill")
            del ctx, pools
            torch.cuda.empty_cache()
    return _with_clocks(rows, spans, sampler)


def sweep_few_long_contexts(reps: int, log) -> list:
    """Decode-only launches over one or four long contexts: every warp streams a slice of the same request, and the
    slices of a (request, KV head) are merged by the units that finish last."""
    import torch

    from . import binding as B
    from .clocks import ClockSampler

    sampler = ClockSampler(0)
    sampler.start()
    spans = []
    dev = torch.device("cuda", 0)
    shape = W.LLAMA
    rows = []
    for lens in ([8192], [65536], [196608], [600000], [16384] * 4, [49152] * 4):
        need = sum(-(-x // shape.page_size) for x in lens) + 64
        batch = W.make_batch(shape, need, lens, 0, 0, W.rng_for(2))
        pools = []
        for layer in range(2):
            t = torch.empty(batch.num_pages * shape.page_elems, dtype=torch.bfloat16, device=dev)
            W.fill_normal_bf16_(t, W.SEED_BASE + 800 + layer)
            pools.append(t)
        ctx = B.Context(shape, batch.num_pages, 1, len(lens), int(batch.decode_pages.shape[0]) + 16)
        q = torch.randn(batch.num_rows, shape.num_q_heads, shape.head_dim, device=dev).to(torch.bfloat16)
        out = torch.empty_like(q)
        t_begin = time.time()
        p50, p99 = _timed(ctx, pools, B.DeviceBatch(batch, dev), q, out, reps)
        B.sw_check_status(ctx)
        spans.append((t_begin, time.time()))
        kv_bytes = sum(lens) * 2 * shape.num_kv_heads * shape.head_dim * 2
        row = {"contexts": lens, "us_p50": p50 / 2e3, "us_p99": p99 / 2e3, "kv_bytes": kv_bytes,
               "gbs": kv_bytes / (p50 / 2e9) / 1e9}
        rows.append(row)
        log(f"contexts {lens}: {row['us_p50']:8.1f} us (p99 {row['us_p99']:.1f}), {kv_bytes / 1e6:.0f} MB of K/V, {row['gbs']:.0f} GB/s")
        del ctx, pools
        torch.cuda.empty_cache()
    return _with_clocks(rows, spans, sampler)


def main(argv=None):
    import argparse
    import sys

    from . import build

    ap = argparse.ArgumentParser(description="cost surface of a named workload: mixed / prefill-only / decode-only launches")
    ap.add_argument("--config", choices=["chat", "mixed", "long", "multichunk", "longcontext"], default="mixed")
    ap.add_argument("--reps", type=int, default=0,
                    help="timed iterations per point; 0 = by the point's duration (200 below 1 ms, 100 below 5 ms, else 30)")
    ap.add_argument("--out", default=None)
    args = ap.parse_args(argv)
    build.build()
    if args.config == "multichunk":
        rows = sweep_multichunk(args.reps, lambda s: print(s, flush=True))
    elif args.config == "longcontext":
        rows = sweep_few_long_contexts(args.reps, lambda s: print(s, flush=True))
    else:
        rows = sweep(args.config, args.reps, lambda s: print(s, flush=True))
    out = args.out or f"cost_surface_{args.config}.json"
    Path(out).parent.mkdir(parents=True, exist_ok=True)
    Path(out).write_text(json.dumps(rows, indent=1))


if __name__ == "__main__":
    main()

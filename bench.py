#!/usr/bin/env python
"""Benchmark of the mixed prefill-chunk + decode attention iteration.

    python bench.py --gpus 1 --steps 20 --warmup 5            # this library
    python bench.py --impl reference --steps 2 --warmup 1     # the CPU oracle, a bounded sample per step

One "step" is one serving iteration on one layer's KV pool: the KV append and the attention of the whole mixed iteration,
which the library runs as ONE launch of its persistent kernel (``sw_mixed_iteration_run``).  Prints ONE JSON line.

Headline workload (the largest single-GPU configuration): the long-context iteration on the Llama-3-8B attention shape
(32 q heads / 8 KV heads, head_dim 128, bf16, 16-token pages): 16 decodes with contexts uniform in [32768, 131072] plus
one prefill chunk of C=4096 tokens at cached-prefix offset 98304 of a 131072-token prompt.  It is tensor-bound (6.7 TFLOP
of chunk prefill against 5.9 GB of K/V), so ``roofline`` reports achieved bf16 TFLOP/s; ``roofline_decode`` is the
decode part timed alone in the same run (HBM GB/s).  ``sweep`` times the other configurations the targets are stated on
(mixed, prefill-only and decode-only launches of each), every window at least 200 ms long with its own clock record.
Data are synthetic (seeded N(0,1) bf16); successive steps use different pools, whose total size exceeds L2.
"""
from __future__ import annotations

import argparse
import dataclasses
import datetime
import json
import math
import os
import subprocess
import sys
import tempfile
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2609_07883_b200 import workloads as W  # noqa: E402
from paper_2609_07883_b200.clocks import ClockSampler  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
MIN_WINDOW_MS = 200.0       # every timed window is repeated until it is at least this long (--min-window-ms)

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of sw_mixed_attn_kernel (KV append fused in) from ncu captures
# of exactly these workloads, keyed by (workload, decodes, chunk, prefix, variant); the summary that holds each figure is
# named beside it.  A point without a capture reports null.
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("long", 16, 4096, 98304, "mixed"): 8_196_000_000,        # profiles/dram_traffic_long_bench.md (mean of two launches)
    ("long", 16, 4096, 98304, "decode_only"): 5_788_000_000,  # profiles/dram_traffic_long_bench.md
    ("chat", 64, 512, 512, "mixed"): 311_723_520,             # profiles/sw_mixed_attn_kernel_chat_bench.md
}


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return json.loads(p.read_text()), "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ---------------------------------------------------------------------------------------------------------------
# workload accounting (algorithmic bytes / flops of one launch)
# ---------------------------------------------------------------------------------------------------------------
def attention_work(batch: W.MixedBatch) -> dict:
    """Decode: 2*Hkv*d*2 bytes per attended token + q in / out out per request.  Chunk prefill: the prompt's K/V once +
    q / out of the chunk rows, and 4*Hq*d flop per unmasked (query, key) pair (masked halves of diagonal tiles and padding
    are not counted).  Append: the new rows read and written once."""
    sh = batch.shape
    P, C, n = batch.prefix_len, batch.chunk_len, batch.num_decode
    ctx = batch.total_decode_ctx
    qo_row = sh.num_q_heads * sh.head_dim * 2 * 2           # q in + o out, bf16
    decode_bytes = ctx * sh.token_bytes + n * qo_row
    prefill_bytes = ((P + C) * sh.token_bytes if C else 0) + C * qo_row
    pairs = C * P + C * (C + 1) // 2
    return {
        "decode_bytes": int(decode_bytes), "prefill_bytes": int(prefill_bytes),
        "attn_bytes": int(decode_bytes + prefill_bytes),
        "append_bytes": int((C + n) * sh.token_bytes * 2),
        "prefill_flops": int(4 * sh.num_q_heads * sh.head_dim * pairs),
        "decode_flops": int(4 * sh.num_q_heads * sh.head_dim * ctx),
        "prefill_pairs": int(pairs), "decode_keys": int(ctx),
    }


WORKLOAD_DEFAULTS = {  # decodes, chunk, prefix, pools rotated
    "chat": (64, 512, 512, 8),
    "mixed": (128, 4096, 28672, 8),
    "long": (16, 4096, 98304, 2),
}
CONTEXTS = {"chat": "U[256,2048]", "mixed": "lognormal(median 2048, sigma 1) clipped to [128,16384]", "long": "U[32768,131072]"}


def make_batch(workload: str, decodes: int, chunk: int, prefix: int, rank: int, room_for_chunk: int = 0) -> W.MixedBatch:
    """The named workload's iteration; the pool holds the live pages plus a little slack.  ``room_for_chunk`` > chunk
    deals prompt pages for a larger chunk as well (so that the same pools serve several chunk sizes)."""
    big = max(chunk, room_for_chunk)
    if workload == "chat":
        b = W.chat_batch(n=decodes, chunk_len=big, prefix_len=prefix, rng=W.rng_for(1, salt=rank))
    elif workload == "mixed":
        b = W.mixed_batch(big, prefix, n=decodes, rng=W.rng_for(2, salt=rank))
    else:
        b = W.long_batch(big, prefix, n=decodes, rng=W.rng_for(3, salt=rank))
    return dataclasses.replace(b, chunk_len=chunk) if big != chunk else b


def variants_of(batch: W.MixedBatch) -> dict:
    """The iteration as it is, its chunk alone and its decodes alone (the profiler of Sec. 5.1 measures all three)."""
    sh = batch.shape
    empty, one = np.zeros(0, np.int32), np.zeros(1, np.int32)
    out = {"mixed": batch}
    if batch.chunk_len > 0 and batch.num_decode > 0:
        out["prefill_only"] = W.MixedBatch(sh, batch.num_pages, batch.prefix_len, batch.chunk_len, batch.prefill_pages, empty,
                                           one, empty)
        out["decode_only"] = W.MixedBatch(sh, batch.num_pages, 0, 0, empty, batch.decode_kv_len, batch.decode_page_indptr,
                                          batch.decode_pages)
    return out


def describe(workload: str, batch: W.MixedBatch) -> str:
    return (f"{workload} iteration, Llama-3-8B attention shape 32/8/128 bf16, 16-token pages: {batch.num_decode} decodes with "
            f"contexts {CONTEXTS[workload]} (total {batch.total_decode_ctx} tokens) + prefill chunk C={batch.chunk_len} at "
            f"prefix {batch.prefix_len}")


# ---------------------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------------------------
ORACLE_KEYS_PER_S_GUESS = 2.0e7   # only sizes the first sample; the rate is measured


class OracleSampler:
    """Times the oracle, as it stands, on random (row, head) pairs of a workload and extrapolates to the whole iteration
    by attended keys.  Large workloads: the sampled rows' pages are drawn into a compact host pool (renumbered page ids,
    seeded N(0,1) content); decode rows then come from one of the requests so that the pool stays small."""

    def __init__(self, batch: W.MixedBatch, seed: int = 1234):
        from oracle import sw_oracle

        self.oracle = sw_oracle
        sh = batch.shape
        rng = np.random.default_rng(seed)
        C, n = batch.chunk_len, batch.num_decode
        self.full = batch
        self.row_keys = np.concatenate([batch.prefix_len + 1 + np.arange(C, dtype=np.int64), batch.decode_kv_len.astype(np.int64)])
        self.total_keys = int(self.row_keys.sum()) * sh.num_q_heads
        total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
        if total_pages * sh.page_elems * 2 <= (1 << 30):
            self.batch, self.rows = batch, np.arange(C + n)
            self.restriction = ""
        else:
            keep = sorted(int(i) for i in rng.choice(n, size=min(n, 1), replace=False)) if n else []
            lens = batch.decode_kv_len[keep] if keep else np.zeros(0, np.int32)
            lists = [batch.decode_pages[batch.decode_page_indptr[i]:batch.decode_page_indptr[i + 1]] for i in keep]
            indptr = np.zeros(len(keep) + 1, np.int32)
            indptr[1:] = np.cumsum([len(x) for x in lists])
            n_dec_pages = int(indptr[-1])
            n_pf = int(batch.prefill_pages.shape[0])
            self.batch = W.MixedBatch(sh, n_dec_pages + n_pf, batch.prefix_len, C, np.arange(n_dec_pages, n_dec_pages + n_pf, dtype=np.int32),
                                      np.asarray(lens, np.int32), indptr, np.arange(n_dec_pages, dtype=np.int32))
            self.rows = np.concatenate([np.arange(C), C + np.arange(len(keep))])   # rows of the compact batch
            self.restriction = f"; decode rows from {len(keep)} of the {n} requests (compact pool of the sampled rows' pages)"
        # q of the compact batch's rows and the pool, seeded N(0,1)
        self.q = W.normal_bf16_bits(rng, self.batch.num_rows, sh.num_q_heads, sh.head_dim)
        self.pool = np.empty(self.batch.num_pages * sh.page_elems, dtype=np.uint16)
        for start in range(0, self.pool.size, 1 << 24):     # in slabs: the conversion's temporaries stay small
            stop = min(self.pool.size, start + (1 << 24))
            self.pool[start:stop] = W.normal_bf16_bits(rng, stop - start)
        self.compact_row_keys = np.concatenate([batch.prefix_len + 1 + np.arange(C, dtype=np.int64),
                                                self.batch.decode_kv_len.astype(np.int64)])
        self.rate = ORACLE_KEYS_PER_S_GUESS

    def sample(self, seconds: float, seed: int):
        """Run the oracle on about ``seconds`` worth of random pairs.  Returns (extrapolated seconds for the whole
        iteration, seconds measured, description)."""
        Hq = self.batch.shape.num_q_heads
        rng = np.random.default_rng(seed)
        order = rng.permutation(len(self.rows) * Hq)
        keys_cum = np.cumsum(self.compact_row_keys[order // Hq])
        budget = max(1.0, seconds * self.rate)
        m = max(1, min(int(np.searchsorted(keys_cum, budget) + 1), len(order)))
        pairs = np.stack([order[:m] // Hq, order[:m] % Hq], axis=1).astype(np.int32)
        sample_keys = int(keys_cum[m - 1])
        t0 = time.perf_counter()
        self.oracle.mixed_attention(self.pool, self.batch, self.q, pairs=pairs)
        dt = time.perf_counter() - t0
        self.rate = sample_keys / max(dt, 1e-6)
        full = dt * self.total_keys / sample_keys
        desc = (f"{m} of {self.full.num_rows * Hq} (row, head) pairs chosen at random = {sample_keys} of {self.total_keys} "
                f"attended keys{self.restriction}; whole-iteration time extrapolated by keys; measured {dt:.2f} s")
        return full, dt, desc

    def threads(self) -> int:
        return self.oracle.num_threads()


# ---------------------------------------------------------------------------------------------------------------
# multi-process plumbing (one process per GPU; replicas only: the path has no exchange step)
# ---------------------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def reduce_max_over_ranks(x, device=None):
    """Element-wise max over ranks of per-rank durations (identity when no process group is initialised).  Accepts a
    number or a list."""
    import torch
    import torch.distributed as dist

    scalar = not isinstance(x, (list, tuple, np.ndarray))
    vals = [float(x)] if scalar else [float(v) for v in x]
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        t = torch.tensor(vals, dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        vals = [float(v) for v in t.tolist()]
    return vals[0] if scalar else vals


def whole_job(us: float, world: int, chunk: int, decodes: int, sharded: bool = False) -> dict:
    """Whole-job numbers from the iteration time of the slowest rank.  N independent replicas: throughputs add up.  One
    iteration sharded by KV heads over N ranks (``sharded``): there is still one iteration's worth of tokens."""
    jobs = 1 if sharded else world
    return {"value": us, "iterations_per_s": jobs / (us * 1e-6), "prefill_tokens_per_s": jobs * chunk / (us * 1e-6),
            "decode_tokens_per_s": jobs * decodes / (us * 1e-6)}


def aggregate_result(per_rank_us: float, world: int, chunk: int, decodes: int, device=None, sharded: bool = False) -> dict:
    """``whole_job`` of the max over ranks of a per-rank iteration time."""
    return whole_job(reduce_max_over_ranks(per_rank_us, device), world, chunk, decodes, sharded)


def spread(us_per_step) -> dict:
    a = np.asarray(us_per_step, dtype=np.float64)
    return {"min": float(a.min()), "median": float(np.median(a)), "max": float(a.max()), "repeats": int(a.size)}


# ---------------------------------------------------------------------------------------------------------------
# one workload on the device
# ---------------------------------------------------------------------------------------------------------------
class DeviceCase:
    """Pools, q / k_new / v_new / out and the device batches of one workload's variants."""

    def __init__(self, B, batch: W.MixedBatch, layers: int, dev, seed: int, max_chunk: int = 0):
        import torch

        self.B, self.batch, self.dev, self.layers = B, batch, dev, layers
        sh = batch.shape
        total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
        self.ctx = B.Context(sh, batch.num_pages, max(batch.chunk_len, max_chunk, 1), max(batch.num_decode, 1), total_pages + 16,
                             device=dev.index)
        self.pools = []
        for layer in range(layers):
            pool = torch.empty(batch.num_pages * sh.page_elems, dtype=torch.bfloat16, device=dev)
            W.fill_normal_bf16_(pool, seed + layer)
            self.pools.append(pool)
        gen = torch.Generator(device=dev)
        gen.manual_seed(seed + 77)
        R = max(batch.chunk_len, max_chunk) + batch.num_decode
        self.q = torch.randn(R, sh.num_q_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
        self.k_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
        self.v_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
        self.out = torch.zeros_like(self.q)

    def stepper(self, batch: W.MixedBatch):
        """step(i) for one variant: KV append + attention in one launch on pool i mod layers.  Decode-only variants take
        the decode rows of q / k_new / v_new (they follow the chunk rows)."""
        B = self.B
        db = B.DeviceBatch(batch, self.dev)
        first = self.batch.chunk_len if batch.chunk_len == 0 and self.batch.chunk_len > 0 else 0
        rows = slice(first, first + batch.num_rows)
        q, k, v, o = self.q[rows], self.k_new[rows], self.v_new[rows], self.out[rows]

        def step(i):
            B.sw_mixed_iteration_run(self.ctx, self.pools[i % self.layers], db, k, v, q, o)

        step.keepalive = db
        return step


def time_window(step, K: int, min_ms: float, sync_all, reduce_max, warmup: int):
    """``warmup`` untimed steps, then the K-step loop, each pass bracketed by CUDA events on the launching stream, repeated
    until the window is at least ``min_ms`` long.  Returns (per-step microseconds of every pass, max over ranks; host time
    stamps of the window)."""
    import torch

    for i in range(warmup):
        step(i)
    sync_all()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for i in range(K):
        step(i)
    c1.record()
    torch.cuda.synchronize()
    est_ms = max(reduce_max(c0.elapsed_time(c1)), 1e-3)
    repeats = int(reduce_max(max(1, math.ceil(min_ms / est_ms))))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    sync_all()
    t0 = time.time()
    ev[0].record()
    for r in range(repeats):
        for i in range(K):
            step(r * K + i)
        ev[r + 1].record()
    sync_all()
    t1 = time.time()
    per_pass_ms = reduce_max([ev[r].elapsed_time(ev[r + 1]) for r in range(repeats)])
    return [ms / K * 1e3 for ms in per_pass_ms], (t0, t1)


def rates(work: dict, us_prefill, us_decode, peaks) -> dict:
    out = {}
    if us_prefill:
        tf = work["prefill_flops"] / (us_prefill * 1e-6) / 1e12
        out.update({"prefill_tflops": tf, "prefill_frac_of_burst": tf / peaks["bf16_tflops"],
                    "prefill_frac_of_sustained": tf / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                    "prefill_frac_of_nominal": tf / NOMINAL_BF16_TFLOPS})
    if us_decode:
        gbs = work["decode_bytes"] / (us_decode * 1e-6) / 1e9
        out.update({"decode_gbs": gbs, "decode_frac_of_measured": gbs / peaks["hbm_gbs"],
                    "decode_frac_of_nominal": gbs / NOMINAL_HBM_GBS})
    return out


# ---------------------------------------------------------------------------------------------------------------
# main legs
# ---------------------------------------------------------------------------------------------------------------
def run_reference(args) -> dict:
    rank, _, _ = dist_env()
    if rank != 0:
        return {}          # under torchrun only rank 0 runs the oracle; the others exit 0 without work
    batch = make_batch(args.workload, args.decodes, args.chunk, args.prefix, 0)
    sampler = OracleSampler(batch)
    times, desc = [], ""
    per_step_s = args.ref_seconds or max(0.5, min(6.0, 150.0 / max(1, args.steps + args.warmup)))
    for step in range(-max(args.warmup, 1), args.steps):
        full, dt, desc = sampler.sample(per_step_s, seed=step + 1000)
        if step >= 0:
            times.append(full)
    us = float(np.mean(times)) * 1e6
    return {
        "impl": "reference", "metric": "mixed_iteration_us", "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args, batch),
        "cpu_baseline": {"value": us, "unit": "us", "cores": sampler.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def workload_config(args, batch) -> dict:
    return {"workload": describe(args.workload, batch), "layers_rotated": args.layers,
            "l2": "inputs larger than L2: step k uses pool k mod layers_rotated",
            "decodes": args.decodes, "chunk": args.chunk, "prefix": args.prefix}


SWEEP = [  # (workload, decodes, chunk, prefix): the configurations the roofline targets are stated on
    ("long", 16, 8192, 98304),
    ("mixed", 128, 4096, 28672),
    ("mixed", 128, 4096, 0),
    ("mixed", 128, 2048, 0),
    ("chat", 64, 512, 512),
]


def run_ours(args) -> dict:
    import torch
    import torch.distributed as dist

    from paper_2609_07883_b200 import build

    rank, local_rank, world = dist_env()
    if rank == 0:
        build.build()
    # one rank per GPU; with fewer GPUs than ranks (a single-GPU check of the N > 1 plumbing with --dist-backend gloo) the
    # ranks share the devices round robin
    gpu = local_rank % max(1, torch.cuda.device_count())
    if world > 1:
        if args.dist_backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", gpu))
        else:
            dist.init_process_group(args.dist_backend)
        dist.barrier()
    from paper_2609_07883_b200 import binding as B

    torch.cuda.set_device(gpu)
    dev = torch.device("cuda", gpu)
    reduce_dev = dev if args.dist_backend == "nccl" else None   # gloo reduces host tensors
    sharded = args.parallel == "heads" and world > 1
    is_default = (args.workload, args.decodes, args.chunk, args.prefix) == ("long",) + WORKLOAD_DEFAULTS["long"][:3]
    do_sweep = world == 1 and not args.no_sweep and is_default
    # the long pools also serve the sweep's C=8192 point: the prompt's page list is dealt for the larger chunk
    batch = make_batch(args.workload, args.decodes, args.chunk, args.prefix, 0 if sharded else rank,
                       room_for_chunk=8192 if do_sweep else 0)
    if sharded:
        # every rank runs the same iteration on its share of the KV heads (and of the query heads that read them)
        from paper_2609_07883_b200 import sharding

        batch = sharding.shard_batch(batch, world)
    work = attention_work(batch)
    peaks, peak_kind = measured_peaks()

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def reduce_max(x):
        return reduce_max_over_ranks(x, reduce_dev)

    sampler = ClockSampler(gpu)
    if rank == 0:
        sampler.start()
    case = DeviceCase(B, batch, args.layers, dev, W.SEED_BASE + 100 + 1000 * rank, max_chunk=8192 if do_sweep else 0)
    variants = variants_of(batch)
    windows = {}   # name -> (per-step us list, (t0, t1))

    # (1) the timed region: K steps of the whole iteration, device-timed, repeated until it is 200 ms long
    step = case.stepper(batch)
    windows["mixed"] = time_window(step, args.steps, args.min_window_ms, sync_all, reduce_max, args.warmup)
    B.sw_check_status(case.ctx)
    launches = args.steps * len(windows["mixed"][0])
    # (2) the decode part and the prefill part alone, same pools, same rotation
    for name in ("decode_only", "prefill_only"):
        if name in variants:
            windows[name] = time_window(case.stepper(variants[name]), args.steps, args.min_window_ms, sync_all, reduce_max, 3)
    B.sw_check_status(case.ctx)
    us = float(np.median(windows["mixed"][0]))
    agg = whole_job(us, world, batch.chunk_len, batch.num_decode, sharded)   # the windows hold the max over ranks already

    # (3) end to end through the host-buffer entry point (pinned host memory, H2D + D2H inside the timed region)
    e2e = None
    if not args.no_e2e:
        hs, keep = B.host_batch_struct(batch)
        R = batch.num_rows
        h_q, h_k, h_v = (t[:R].cpu().pin_memory() for t in (case.q, case.k_new, case.v_new))
        h_out = torch.empty_like(h_q).pin_memory()
        e2e_steps = max(3, min(args.steps, 200))
        for i in range(max(2, min(args.steps, 20))):    # the first calls run slower: pinned-copy paths and clocks settle
            B.sw_mixed_iteration_host(case.ctx, case.pools[i % args.layers], hs, h_q, h_k, h_v, h_out)
        sync_all()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            B.sw_mixed_iteration_host(case.ctx, case.pools[i % args.layers], hs, h_q, h_k, h_v, h_out)
        torch.cuda.synchronize()
        e2e_us = reduce_max((time.perf_counter() - t0) / e2e_steps * 1e6)
        total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
        page_entries = total_pages + 2 * batch.num_decode + 1
        e2e = {"value": e2e_us, "unit": "us",
               "h2d_bytes_per_step": int(h_q.numel() * 2 + h_k.numel() * 2 * 2 + page_entries * 4),
               "d2h_bytes_per_step": int(h_out.numel() * 2)}
        B.sw_check_status(case.ctx)

    # (4) the other configurations the targets are stated on (one GPU, default workload only)
    sweep_rows = []
    if do_sweep:
        cases = {("long", 16, 98304): case}
        for (wl, n, C, P) in SWEEP:
            key = (wl, n, P)
            if key not in cases:
                room = max(c for (w2, n2, c, p2) in SWEEP if (w2, n2, p2) == key)
                b0 = make_batch(wl, n, room, P, rank)
                cases[key] = DeviceCase(B, b0, WORKLOAD_DEFAULTS[wl][3], dev, W.SEED_BASE + 300 + 7 * len(cases), max_chunk=room)
            c = cases[key]
            b = dataclasses.replace(c.batch, chunk_len=C)
            row = {"workload": describe(wl, b), "decodes": n, "chunk": C, "prefix": P, "layers_rotated": c.layers}
            w = attention_work(b)
            tw = {}
            for name, vb in variants_of(b).items():
                per_step, span = time_window(c.stepper(vb), args.steps, args.min_window_ms, sync_all, reduce_max, 3)
                row[name + "_us"] = spread(per_step)
                tw[name] = (per_step, span)
            B.sw_check_status(c.ctx)
            row.update(rates(w, row.get("prefill_only_us", {}).get("median"), row.get("decode_only_us", {}).get("median"), peaks))
            row["mixed_vs_sum"] = row["mixed_us"]["median"] / (row["prefill_only_us"]["median"] + row["decode_only_us"]["median"])
            row["prefill_tokens_per_s"] = C / (row["mixed_us"]["median"] * 1e-6)
            row["decode_tokens_per_s"] = n / (row["mixed_us"]["median"] * 1e-6)
            row["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get((wl, n, C, P, "mixed"))
            row["_spans"] = {k: v[1] for k, v in tw.items()}
            sweep_rows.append(row)
    if rank == 0:
        sampler.stop()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return {}
    for row in sweep_rows:
        spans = row.pop("_spans")
        row["clocks"] = sampler.window(min(s[0] for s in spans.values()), max(s[1] for s in spans.values()))

    # roofline of the dominant kernel: one launch per step, algorithmic work per launch / average launch duration
    clocks = sampler.window(*windows["mixed"][1])
    launch_bytes = work["attn_bytes"] + work["append_bytes"]
    tensor_bound = work["prefill_flops"] / (NOMINAL_BF16_TFLOPS * 1e12) > launch_bytes / (NOMINAL_HBM_GBS * 1e9)
    kernel = f"sw_mixed_attn_kernel<{batch.shape.head_dim}, false> (one prefill chunk; KV append fused in)"
    key = (args.workload, args.decodes, args.chunk, args.prefix)
    if tensor_bound:
        tf = work["prefill_flops"] / (us * 1e-6) / 1e12
        sustained = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        roofline = {"bound": "tensor", "achieved": tf, "peak": sustained, "unit": "TFLOP/s", "frac": tf / sustained,
                    "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(key + ("mixed",)),
                    "peak_kind": f"of {peak_kind} (cuBLAS bf16, sustained figure: the launch is timed inside a loop of "
                                 f"{launches} launches that sits at the power cap)",
                    "frac_of_burst": tf / peaks["bf16_tflops"], "frac_of_nominal": tf / NOMINAL_BF16_TFLOPS,
                    "kernel": kernel, "algorithmic_flops_per_launch": work["prefill_flops"],
                    "algorithmic_bytes_per_launch": launch_bytes,
                    "note": "flops of the chunk prefill only (4*Hq*d per unmasked pair); the same launch also streams the "
                            "decodes' K/V"}
    else:
        gbs = launch_bytes / (us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                    "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(key + ("mixed",)), "peak_kind": f"of {peak_kind}",
                    "frac_of_nominal": gbs / NOMINAL_HBM_GBS, "kernel": kernel, "algorithmic_bytes_per_launch": launch_bytes}
    result = {
        "metric": "mixed_iteration_us", "value": us, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "strong" if sharded else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(args, batch),
        "us_per_step": spread(windows["mixed"][0]), "timed_steps": launches,
        "iterations_per_s": agg["iterations_per_s"],
        "prefill_tokens_per_s": agg["prefill_tokens_per_s"],
        "decode_tokens_per_s": agg["decode_tokens_per_s"],
        "roofline": roofline,
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if "decode_only" in windows:
        d_us = float(np.median(windows["decode_only"][0]))
        p_us = float(np.median(windows["prefill_only"][0]))
        r = rates(work, p_us, d_us, peaks)
        result["roofline_decode"] = {"bound": "hbm", "achieved": r["decode_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                     "frac": r["decode_frac_of_measured"], "frac_of_nominal": r["decode_frac_of_nominal"],
                                     "peak_kind": f"of {peak_kind}", "us_per_step": spread(windows["decode_only"][0]),
                                     "algorithmic_bytes_per_launch": work["decode_bytes"],
                                     "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(key + ("decode_only",)),
                                     "clocks": sampler.window(*windows["decode_only"][1]),
                                     "what": "the iteration's decodes alone (same pools, same launch path)"}
        result["prefill_only"] = {"us_per_step": spread(windows["prefill_only"][0]), "tflops": r["prefill_tflops"],
                                  "frac_of_burst": r["prefill_frac_of_burst"], "frac_of_sustained": r["prefill_frac_of_sustained"],
                                  "frac_of_nominal": r["prefill_frac_of_nominal"],
                                  "clocks": sampler.window(*windows["prefill_only"][1])}
        result["mixed_vs_sum"] = us / (d_us + p_us)
    if e2e:
        result["e2e"] = e2e
    if sweep_rows:
        result["sweep"] = sweep_rows
    if world == 1 and not args.no_cpu_baseline:
        osamp = OracleSampler(batch)
        osamp.sample(1.0, seed=1)                      # measures the oracle's rate on this machine
        full, dt, desc = osamp.sample(args.cpu_seconds, seed=2)
        result["cpu_baseline"] = {"value": full * 1e6, "unit": "us", "cores": osamp.threads(), "kind": "oracle", "sample": desc}
    if world > 1:
        dist.destroy_process_group()
    return result


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long", choices=sorted(WORKLOAD_DEFAULTS))
    ap.add_argument("--decodes", type=int, default=None)
    ap.add_argument("--chunk", type=int, default=None)
    ap.add_argument("--prefix", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None, help="pools rotated through (working set > L2)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU time given to the oracle sample of cpu_baseline")
    ap.add_argument("--ref-seconds", type=float, default=0.0,
                    help="--impl reference: CPU time per step's oracle sample (default: sized so that the run ends in minutes)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="time the named workload only")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--min-window-ms", type=float, default=MIN_WINDOW_MS,
                    help="every timed window repeats its K-step loop until it is this long (0: once; for profiler captures)")
    ap.add_argument("--dist-backend", default="nccl", choices=["nccl", "gloo"],
                    help="N > 1: process-group backend (gloo lets several ranks share one GPU to check the plumbing)")
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: independent replicas (default) or one iteration sharded by KV heads, no collective either way")
    args = ap.parse_args()
    dn, dc, dp, dl = WORKLOAD_DEFAULTS[args.workload]
    args.decodes = dn if args.decodes is None else args.decodes
    args.chunk = dc if args.chunk is None else args.chunk
    args.prefix = dp if args.prefix is None else args.prefix
    args.layers = dl if args.layers is None else args.layers
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    res = run_reference(args) if args.impl == "reference" else run_ours(args)
    if res:
        print(json.dumps(res))


if __name__ == "__main__":
    main()

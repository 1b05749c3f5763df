#!/usr/bin/env python
"""Benchmark of the mixed prefill-chunk + decode attention iteration (one "step" = KV append + the single
attention launch of one iteration, on one layer's pool of a rotating layer stack).

    python bench.py --gpus 1 --steps 50 --warmup 5            # this library
    python bench.py --impl reference --steps 2 --warmup 1     # the CPU oracle, bounded sample per step

Prints ONE JSON line.  Workload: the chat-like iteration on the Llama-3-8B attention shape (32 q heads / 8 KV
heads, head_dim 128, bf16, 16-token pages): 64 decodes with contexts uniform in [256, 2048] plus one prefill
chunk C=512 at prefix 512 of a 1024-token prompt.  Data are synthetic (seeded N(0,1) bf16).
"""
from __future__ import annotations

import argparse
import json
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

# dram__bytes_read.sum + dram__bytes_write.sum of one sw_mixed_attn_kernel<128> launch of the default workload, from the
# ncu capture summarised in profiles/sw_mixed_attn_kernel_chat_bench.md (298.8 MB read + 12.6 MB written; the launch
# includes the fused KV append)
NCU_TRAFFIC_DEFAULT_WORKLOAD = 311_881_984
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return json.loads(p.read_text()), "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ---------------------------------------------------------------------------------------------------------------
# workload accounting (algorithmic bytes / flops of one attention launch)
# ---------------------------------------------------------------------------------------------------------------
def attention_work(batch: W.MixedBatch) -> dict:
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


WORKLOAD_DEFAULTS = {  # decodes, chunk, prefix
    "chat": (64, 512, 512),
    "mixed": (128, 4096, 28672),
    "long": (16, 4096, 98304),
}


def make_workload(args, rank: int) -> W.MixedBatch:
    """chat: contexts U[256, 2048]; mixed: lognormal(median 2048, sigma 1) clipped to [128, 16384];
    long: U[32768, 131072].  The pool holds the live pages plus a little slack."""
    if args.workload == "chat":
        return W.chat_batch(n=args.decodes, chunk_len=args.chunk, prefix_len=args.prefix, rng=W.rng_for(1, salt=rank))
    if args.workload == "mixed":
        return W.mixed_batch(args.chunk, args.prefix, n=args.decodes, rng=W.rng_for(2, salt=rank))
    return W.long_batch(args.chunk, args.prefix, n=args.decodes, rng=W.rng_for(3, salt=rank))


# ---------------------------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        try:
            for line in open(self.path).read().splitlines():
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    smax.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [x for x in sm if x > 0.5 * max(sm)]
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------------------------
def oracle_sample_time(batch: W.MixedBatch, tensors: dict, budget_keys: int, seed: int = 0):
    """Time the oracle, as it stands, on a random sample of (row, head) pairs holding about `budget_keys` attended
    keys.  Returns (extrapolated seconds for the whole iteration, seconds measured, sample description, threads)."""
    from oracle import sw_oracle

    sh = batch.shape
    C, n, Hq = batch.chunk_len, batch.num_decode, sh.num_q_heads
    row_keys = np.concatenate([batch.prefix_len + 1 + np.arange(C, dtype=np.int64),
                               batch.decode_kv_len.astype(np.int64)])
    total_keys = int(row_keys.sum()) * Hq
    rng = np.random.default_rng(seed)
    order = rng.permutation((C + n) * Hq)
    keys_cum = np.cumsum(row_keys[order // Hq])
    m = int(np.searchsorted(keys_cum, budget_keys) + 1)
    m = max(1, min(m, len(order)))
    pairs = np.stack([order[:m] // Hq, order[:m] % Hq], axis=1).astype(np.int32)
    sample_keys = int(keys_cum[m - 1])
    t0 = time.perf_counter()
    sw_oracle.mixed_attention(tensors["pool"], batch, tensors["q"], pairs=pairs)
    dt = time.perf_counter() - t0
    full = dt * total_keys / sample_keys
    desc = (f"{m} of {(C + n) * Hq} (row, head) pairs chosen at random = {sample_keys} of {total_keys} attended keys; "
            f"whole-iteration time extrapolated by keys")
    return full, dt, desc, sw_oracle.num_threads()


def host_tensors_for(batch: W.MixedBatch, seed: int) -> dict:
    rng = np.random.default_rng(seed)
    return W.host_tensors(batch, rng, with_pool=True)


# ---------------------------------------------------------------------------------------------------------------
# multi-process plumbing (one process per GPU; replicas only: the path has no exchange step)
# ---------------------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def reduce_max_over_ranks(x: float, device=None) -> float:
    """max over ranks of a per-rank duration (identity when no process group is initialised)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_result(per_rank_us: float, world: int, chunk: int, decodes: int, device=None, sharded: bool = False) -> dict:
    """Whole-job numbers.  N independent replicas: the iteration time is the slowest rank's, throughputs add up.  One
    iteration sharded by KV heads over N ranks (``sharded``): the iteration ends with its slowest rank and there is still
    one iteration's worth of tokens."""
    us = reduce_max_over_ranks(per_rank_us, device)
    jobs = 1 if sharded else world
    return {"value": us, "iterations_per_s": jobs / (us * 1e-6), "prefill_tokens_per_s": jobs * chunk / (us * 1e-6),
            "decode_tokens_per_s": jobs * decodes / (us * 1e-6)}


# ---------------------------------------------------------------------------------------------------------------
# main legs
# ---------------------------------------------------------------------------------------------------------------
def run_reference(args) -> dict:
    rank, _, _ = dist_env()
    if rank != 0:
        return {}          # under torchrun only rank 0 runs the oracle; the others exit 0 without work
    batch = make_workload(args, 0)
    tensors = host_tensors_for(batch, 1234)
    times = []
    desc, threads = "", 1
    for step in range(-args.warmup, args.steps):
        full, dt, desc, threads = oracle_sample_time(batch, tensors, args.ref_budget_keys, seed=step + 1000)
        if step >= 0:
            times.append(full)
    us = float(np.mean(times)) * 1e6
    return {
        "impl": "reference", "metric": "mixed_iteration_us", "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args, batch),
        "cpu_baseline": {"value": us, "unit": "us", "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def workload_config(args, batch) -> dict:
    dist = {"chat": "U[256,2048]", "mixed": "lognormal(median 2048, sigma 1) clipped to [128,16384]",
            "long": "U[32768,131072]"}[args.workload]
    return {"workload": f"{args.workload} iteration, Llama-3-8B attention shape 32/8/128 bf16, 16-token pages: {args.decodes} decodes "
                        f"with contexts {dist} (total {batch.total_decode_ctx} tokens) + prefill chunk C={args.chunk} at "
                        f"prefix {args.prefix}",
            "layers_rotated": args.layers, "l2": "inputs larger than L2: step k uses pool k mod layers",
            "decodes": args.decodes, "chunk": args.chunk, "prefix": args.prefix}


def run_ours(args) -> dict:
    import torch
    import torch.distributed as dist

    from paper_2609_07883_b200 import build

    rank, local_rank, world = dist_env()
    if rank == 0:
        build.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2609_07883_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    sharded = args.parallel == "heads" and world > 1
    batch = make_workload(args, 0 if sharded else rank)
    if sharded:
        # every rank runs the same iteration on its share of the KV heads (and of the query heads that read them)
        from paper_2609_07883_b200 import sharding

        batch = sharding.shard_batch(batch, world)
    sh = batch.shape
    work = attention_work(batch)
    total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
    ctx = B.Context(sh, batch.num_pages, batch.chunk_len, batch.num_decode, total_pages + 16, device=local_rank)
    dbatch = B.DeviceBatch(batch, dev)
    pools = []
    for layer in range(args.layers):
        pool = torch.empty(batch.num_pages * sh.page_elems, dtype=torch.bfloat16, device=dev)
        W.fill_normal_bf16_(pool, W.SEED_BASE + 100 + layer + 1000 * rank)
        pools.append(pool)
    gen = torch.Generator(device=dev)
    gen.manual_seed(W.SEED_BASE + 7 + rank)
    R = batch.num_rows
    q = torch.randn(R, sh.num_q_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    k_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    v_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    out = torch.zeros_like(q)

    def step(i):
        pool = pools[i % args.layers]
        B.sw_mixed_iteration_run(ctx, pool, dbatch, k_new, v_new, q, out)  # KV append + attention, one launch

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def reduce_max(x: float) -> float:
        return reduce_max_over_ranks(x, dev)

    # clocks are sampled from before the warm-up to after the last timed loop (nvidia-smi needs a moment to start)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.4)
    for i in range(args.warmup):
        step(i)
    sync_all()
    B.sw_check_status(ctx)
    # (1) the timed region: K steps, device-timed
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    sync_all()
    ms_local = e0.elapsed_time(e1)
    agg = aggregate_result(ms_local / args.steps * 1e3, world, batch.chunk_len, batch.num_decode, dev, sharded)
    ms_total = agg["value"] * args.steps / 1e3
    # (2) the attention launch alone (dominant kernel) for the roofline, same stream, same rotation
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for i in range(args.steps):
        B.sw_mixed_attn_run(ctx, pools[i % args.layers], dbatch, q, out)
    a1.record()
    torch.cuda.synchronize()
    attn_ms = a0.elapsed_time(a1) / args.steps
    # (3) end to end through the host-buffer entry point (pinned host memory, H2D + D2H inside the timed region)
    hs, keep = B.host_batch_struct(batch)
    h_q, h_k, h_v = (t.cpu().pin_memory() for t in (q, k_new, v_new))
    h_out = torch.empty_like(h_q).pin_memory()
    # (the first hundred or so calls run slower than the steady state: pinned-copy paths and clocks settle)
    e2e_steps = max(3, min(args.steps, 200))
    for i in range(max(2, min(args.steps, 100))):
        B.sw_mixed_iteration_host(ctx, pools[i % args.layers], hs, h_q, h_k, h_v, h_out)
    sync_all()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        B.sw_mixed_iteration_host(ctx, pools[i % args.layers], hs, h_q, h_k, h_v, h_out)
    torch.cuda.synchronize()
    e2e_us = reduce_max((time.perf_counter() - t0) / e2e_steps * 1e6)
    clocks = sampler.stop() if rank == 0 else {}
    B.sw_check_status(ctx)

    page_entries = total_pages + 2 * batch.num_decode + 1
    h2d = int(q.numel() * 2 + k_new.numel() * 2 * 2 + page_entries * 4)
    d2h = int(out.numel() * 2)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return {}

    us = ms_total / args.steps * 1e3
    peaks, peak_kind = measured_peaks()
    # A step is ONE launch of sw_mixed_attn_kernel (append fused in): its algorithmic bytes are the attention's plus the
    # new rows read and written once, its duration the launch-to-launch time of the timed region.
    sh = batch.shape
    append_bytes = batch.num_rows * sh.num_kv_heads * sh.head_dim * 2 * 2 * 2
    launch_bytes = work["attn_bytes"] + append_bytes
    achieved_gbs = launch_bytes / (us * 1e-6) / 1e9
    is_default = (args.workload, args.decodes, args.chunk, args.prefix) == ("chat",) + WORKLOAD_DEFAULTS["chat"]
    traffic = NCU_TRAFFIC_DEFAULT_WORKLOAD if is_default else None
    result = {
        "metric": "mixed_iteration_us", "value": us, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": False,
        "scaling": "strong" if sharded else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(args, batch),
        "iterations_per_s": agg["iterations_per_s"],
        "prefill_tokens_per_s": agg["prefill_tokens_per_s"],
        "decode_tokens_per_s": agg["decode_tokens_per_s"],
        "attn_launch_us": attn_ms * 1e3,
        "roofline": {"bound": "hbm", "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved_gbs / peaks["hbm_gbs"], "traffic": traffic, "peak_kind": f"of {peak_kind}",
                     "kernel": "sw_mixed_attn_kernel<128, false> (one prefill chunk; KV append fused in)", "algorithmic_bytes_per_launch": launch_bytes,
                     "attention_only_launch_gbs": work["attn_bytes"] / (attn_ms * 1e-3) / 1e9,
                     "frac_of_nominal_8TBs": achieved_gbs / NOMINAL_HBM_GBS,
                     "prefill_tflops": work["prefill_flops"] / (us * 1e-6) / 1e12},
        "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": args.steps,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        tensors = host_tensors_for(batch, 1234)
        full, dt, desc, threads = oracle_sample_time(batch, tensors, args.cpu_budget_keys)
        result["cpu_baseline"] = {"value": full * 1e6, "unit": "us", "cores": threads, "kind": "oracle",
                                  "sample": desc + f"; measured {dt:.2f} s"}
    if world > 1:
        dist.destroy_process_group()
    return result


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="chat", choices=sorted(WORKLOAD_DEFAULTS))
    ap.add_argument("--decodes", type=int, default=None)
    ap.add_argument("--chunk", type=int, default=None)
    ap.add_argument("--prefix", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None, help="pools rotated through (working set > L2)")
    ap.add_argument("--cpu-budget-keys", type=int, default=1_000_000_000)
    ap.add_argument("--ref-budget-keys", type=int, default=1_000_000_000)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "heads"],
                    help="N > 1: independent replicas (default) or one iteration sharded by KV heads, no collective either way")
    args = ap.parse_args()
    dn, dc, dp = WORKLOAD_DEFAULTS[args.workload]
    args.decodes = dn if args.decodes is None else args.decodes
    args.chunk = dc if args.chunk is None else args.chunk
    args.prefix = dp if args.prefix is None else args.prefix
    if args.layers is None:
        args.layers = 8 if args.workload == "chat" else 2
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    res = run_reference(args) if args.impl == "reference" else run_ours(args)
    if res:
        print(json.dumps(res))


if __name__ == "__main__":
    main()

"""The event-driven simulator study (Sec. 4): policies compared under the analytic iteration cost, on the CPU.

The loop is the serving loop of ``serving.run_trace`` (one decode token per active request and at most one prefill
chunk per iteration, arrivals eligible at the end of the iteration, oldest-first queue) with the virtual clock advanced
by the analytic cost model ``T(n, c)`` of Sec. 4.1 instead of measured device time.  The controller is the library's
``sw_choose_chunk`` (Algorithm 1) on an exact table of the same model, so SLOWeave's predictions are exact here, as in
the paper's simulator.  Policies: full-prompt prefill, fixed chunks, SLOWeave with ``C_max = 4096`` (Sec. 4.3).

The paper does not state the log-normal sigmas, the clipping ranges, the burst parameters or the seeds of its traces
(``workloads.study_trace`` states the values chosen here), so the numbers of Tables 3-4 cannot be reproduced digit for
digit; the study shows the same trends on traces of the stated shape.

    python -m paper_2609_07883_b200.simulate --out simulator_study.json
"""
from __future__ import annotations

import argparse
import json
import time
from pathlib import Path

import numpy as np

from . import workloads as W

MS = 1_000_000
FULL = 1 << 30  # a "fixed chunk" larger than any prompt: full-prompt prefill


def analytic_cost_ns(n: int, c: int) -> int:
    """Iteration cost of the default model (Sec. 4.1), in integer nanoseconds:
    T(n, c) = 0.35 + 1[n > 0] (0.90 + 0.055 n) + 1[c > 0] (0.40 + 0.006 c) ms."""
    t = 350_000
    if n > 0:
        t += 900_000 + 55_000 * n
    if c > 0:
        t += 400_000 + 6_000 * c
    return t


def analytic_table(max_decode: int, c_max: int, quantum: int):
    """Exact table of the model on every decode count 1..max_decode and every multiple of the chunk quantum."""
    from . import binding as B

    n_values = list(range(1, max_decode + 1))
    chunk_grid = list(range(0, c_max + 1, quantum))
    if chunk_grid[-1] != c_max:
        chunk_grid.append(c_max)
    cost = np.array([[analytic_cost_ns(n, c) for c in chunk_grid] for n in n_values], dtype=np.int64)
    return B.CostTable(n_values, [1 << 40], [1 << 30], chunk_grid, cost.reshape(len(n_values), 1, 1, -1))


POLICIES = {"full": f"fixed:{FULL}", "fixed-64": "fixed:64", "fixed-256": "fixed:256", "fixed-1024": "fixed:1024",
            "sloweave": "sloweave", "sloweave-8": "sloweave"}
# "sloweave-8" admits up to eight pending prompts per iteration by first fit (Sec. 3.3, "Prefill batching"); the
# paper's own study admits one, so it is not part of the default policy list.
MAX_PREFILLS = {"sloweave-8": 8}
DEFAULT_POLICIES = ["full", "fixed-64", "fixed-256", "fixed-1024", "sloweave"]


def run_one(workload: str, policy: str, tpot_ms: float, seed: int, table, num_requests: int, c_max: int, quantum: int,
            max_decode: int) -> dict:
    from . import serving

    trace = W.study_trace(workload, seed, num_requests)
    res = serving.run_trace(trace, tpot_ms, table, lambda b: analytic_cost_ns(b.num_decode, b.chunk_len), W.LLAMA,
                            1 << 21, policy=POLICIES[policy], c_max=c_max, margin_ppm=0, quantum=quantum,
                            max_decode=max_decode, page_tables=False, ttft_slo_ms=W.STUDY[workload]["ttft_slo_ms"],
                            max_prefills=MAX_PREFILLS.get(policy, 1))
    res["workload"], res["policy"], res["seed"] = workload, policy, seed
    return res


def study(workloads, policies, tpots, seeds, num_requests: int = 1000, c_max: int = 4096, quantum: int = 16,
          max_decode: int = 1024, log=None) -> dict:
    """Runs every (workload, TPOT, policy, seed); returns the per-seed rows and their means over the seeds."""
    table = analytic_table(max_decode, c_max, quantum)
    rows, means = [], []
    keys = ("ttft_ms_p99", "tpot_ms_p99_of_request_p99", "throughput_rps", "slo_attainment", "goodput_rps",
            "deadline_misses_with_chunk", "mean_chunk")
    for wl in workloads:
        for tpot in tpots:
            for pol in policies:
                t0 = time.time()
                per_seed = [run_one(wl, pol, tpot, s, table, num_requests, c_max, quantum, max_decode) for s in seeds]
                rows += per_seed
                m = {"workload": wl, "tpot_ms": tpot, "policy": pol, "seeds": len(per_seed)}
                m.update({k: float(np.mean([r[k] for r in per_seed])) for k in keys})
                means.append(m)
                if log:
                    log(f"{wl:7s} TPOT {tpot:4.0f} ms {pol:10s}  P99 TTFT {m['ttft_ms_p99']:8.0f} ms  P99 TPOT "
                        f"{m['tpot_ms_p99_of_request_p99']:6.1f} ms  SLO {100 * m['slo_attainment']:5.1f} %  goodput "
                        f"{m['goodput_rps']:6.1f} req/s  ({time.time() - t0:.0f} s)")
    return {"requests": num_requests, "c_max": c_max, "quantum": quantum, "means": means, "rows": rows}


def ratios(means) -> list:
    """SLOWeave's goodput over the strongest static policy, per workload and TPOT (the quantity of Table 4)."""
    out = []
    for wl in sorted({m["workload"] for m in means}):
        for tpot in sorted({m["tpot_ms"] for m in means}):
            cell = {m["policy"]: m["goodput_rps"] for m in means if m["workload"] == wl and m["tpot_ms"] == tpot}
            static = {k: v for k, v in cell.items() if not k.startswith("sloweave")}
            if "sloweave" not in cell or not static:
                continue
            best = max(static, key=static.get)
            out.append({"workload": wl, "tpot_ms": tpot, "sloweave": cell["sloweave"], "best_static": best,
                        "best_static_goodput": static[best],
                        "ratio": cell["sloweave"] / static[best] if static[best] > 0 else float("inf")})
    return out


def main(argv=None):
    from . import build

    ap = argparse.ArgumentParser(description="simulator study: policies under the analytic cost model (CPU only)")
    ap.add_argument("--workloads", nargs="+", default=["chat", "mixed", "long", "bursty"], choices=sorted(W.STUDY))
    ap.add_argument("--policies", nargs="+", default=DEFAULT_POLICIES, choices=list(POLICIES))
    ap.add_argument("--tpot-ms", type=float, nargs="+", default=[10.0, 25.0, 50.0])
    ap.add_argument("--seeds", type=int, default=5)
    ap.add_argument("--requests", type=int, default=1000)
    ap.add_argument("--out", default="simulator_study.json")
    args = ap.parse_args(argv)
    build.build()
    res = study(args.workloads, args.policies, args.tpot_ms, list(range(args.seeds)), args.requests,
                log=lambda s: print(s, flush=True))
    res["ratios"] = ratios(res["means"])
    for r in res["ratios"]:
        print(f"{r['workload']:7s} TPOT {r['tpot_ms']:4.0f} ms: SLOWeave {r['sloweave']:6.1f} vs {r['best_static']:10s} "
              f"{r['best_static_goodput']:6.1f} req/s = {r['ratio']:.2f}x")
    Path(args.out).parent.mkdir(parents=True, exist_ok=True)
    Path(args.out).write_text(json.dumps(res))


if __name__ == "__main__":
    main()

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


def measure_table(ctx, pools, shape: W.AttnShape, num_pages: int, n_grid, ctx_grid, prefix_grid, chunk_grid,
                  reps: int = 10, warmup: int = 2, seed: int = W.SEED_BASE + 40, progress=None) -> dict:
    """Probe every grid point.  ``ctx`` is a binding.Context big enough for the largest point; ``pools`` the layer
    stack (list of device tensors).  Returns a plain dict (JSON-serialisable) with P50 and P99 per point."""
    import torch

    from . import binding as B

    dev = pools[0].device
    rng = np.random.default_rng(seed)
    max_rows = max(chunk_grid) + max(n_grid)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    q = torch.randn(max_rows, shape.num_q_heads, shape.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    out = torch.empty_like(q)
    shape4 = (len(n_grid), len(ctx_grid), len(prefix_grid), len(chunk_grid))
    p50 = np.zeros(shape4, dtype=np.int64)
    p99 = np.zeros(shape4, dtype=np.int64)
    t0 = time.time()
    for a, n in enumerate(n_grid):
        for b, ctx_total in enumerate(ctx_grid):
            for c_i, prefix in enumerate(prefix_grid):
                for e, chunk in enumerate(chunk_grid):
                    if n == 0 and chunk == 0:
                        continue
                    if chunk == 0 and c_i > 0:      # the decode-only plane does not depend on the prefix
                        p50[a, b, c_i, e], p99[a, b, c_i, e] = p50[a, b, 0, e], p99[a, b, 0, e]
                        continue
                    batch = probe_batch(shape, num_pages, int(n), int(ctx_total), int(prefix), int(chunk), rng)
                    db = B.DeviceBatch(batch, dev)
                    m, h, _ = B.sw_cost_probe(ctx, pools, db, q, out, warmup=warmup, reps=reps)
                    p50[a, b, c_i, e], p99[a, b, c_i, e] = m, h
        if progress:
            progress(f"n={n}: {time.time() - t0:.1f}s")
    B.sw_check_status(ctx)
    return {"n_grid": [int(x) for x in n_grid], "ctx_grid": [int(x) for x in ctx_grid],
            "prefix_grid": [int(x) for x in prefix_grid], "chunk_grid": [int(x) for x in chunk_grid],
            "layers": len(pools), "reps": reps, "warmup": warmup, "p50_ns": p50.tolist(), "p99_ns": p99.tolist(),
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

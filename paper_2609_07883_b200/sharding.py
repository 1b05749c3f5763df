"""KV-head sharding of the mixed iteration over several GPUs (the tensor-parallel setting of Sec. 5.2).

Attention is independent per KV head: rank r of N keeps KV heads [r * Hkv / N, (r + 1) * Hkv / N) of every page and
computes the query heads that read them; no rank needs another rank's K/V, so the data path has no collective.  What
the ranks must share is the controller's view: every rank has to choose the same chunk, so the cost table is the
element-wise maximum of the ranks' measurements (an iteration ends when its slowest rank does).

Slicing helpers work on host arrays (bf16 bits) and on torch tensors alike; page tables, lengths and row order are the
same on every rank.
"""
from __future__ import annotations

import dataclasses

import numpy as np

from . import workloads as W


def shard_shape(shape: W.AttnShape, world: int) -> W.AttnShape:
    if world < 1 or shape.num_kv_heads % world:
        raise ValueError(f"{shape.num_kv_heads} KV heads cannot be shared out among {world} ranks")
    return W.AttnShape(shape.num_q_heads // world, shape.num_kv_heads // world, shape.head_dim, shape.page_size)


def shard_batch(batch: W.MixedBatch, world: int) -> W.MixedBatch:
    """The same iteration (same page tables and lengths) on a rank's share of the heads."""
    return dataclasses.replace(batch, shape=shard_shape(batch.shape, world))


def kv_head_range(shape: W.AttnShape, rank: int, world: int):
    per = shard_shape(shape, world).num_kv_heads
    return rank * per, (rank + 1) * per


def shard_rows(x, shape: W.AttnShape, rank: int, world: int, kind: str):
    """A rank's heads of q / out (``kind="q"``, [rows][Hq][d]) or of k_new / v_new (``kind="kv"``, [rows][Hkv][d])."""
    lo, hi = kv_head_range(shape, rank, world)
    if kind == "q":
        lo, hi = lo * shape.group, hi * shape.group
    heads = shape.num_q_heads if kind == "q" else shape.num_kv_heads
    v = x.reshape(-1, heads, shape.head_dim)
    part = v[:, lo:hi, :]
    return part.contiguous() if hasattr(part, "contiguous") else np.ascontiguousarray(part)


def shard_pool(pool, shape: W.AttnShape, rank: int, world: int):
    """A rank's heads of a pool laid out [page][K|V][Hkv][slot][d] (flat or shaped), as a flat array."""
    lo, hi = kv_head_range(shape, rank, world)
    v = pool.reshape(-1, 2, shape.num_kv_heads, shape.page_size, shape.head_dim)
    part = v[:, :, lo:hi]
    part = part.contiguous() if hasattr(part, "contiguous") else np.ascontiguousarray(part)
    return part.reshape(-1)


def gather_heads(parts, kind_heads_axis: int = 1):
    """Concatenates the ranks' [rows][heads_r][d] outputs along the head axis (rank order = head order)."""
    if hasattr(parts[0], "contiguous"):
        import torch

        return torch.cat(list(parts), dim=kind_heads_axis)
    return np.concatenate(list(parts), axis=kind_heads_axis)


def reduce_table_max(table: dict, group=None) -> dict:
    """Element-wise maximum over the ranks of a measured cost table (``profiler.measure_table`` output): the table every
    rank hands to the controller.  Needs an initialised ``torch.distributed`` process group (gloo or nccl); with a single
    process it returns the table unchanged."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return table
    out = dict(table)
    backend = dist.get_backend(group)
    dev = torch.device("cuda", torch.cuda.current_device()) if backend == "nccl" else torch.device("cpu")
    for key in ("p50_ns", "p99_ns"):
        t = torch.tensor(table[key], dtype=torch.int64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
        out[key] = t.cpu().tolist()
    out["ranks_reduced"] = dist.get_world_size(group)
    return out

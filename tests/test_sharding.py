"""KV-head sharding: the slices are exact partitions (CPU, against the oracle run head by head), the ranks' cost tables
reduce to their maximum (gloo, world size 2), and on a GPU the ranks' outputs put side by side equal the unsharded run."""
import os
import subprocess
import sys
import textwrap

import numpy as np
import pytest

from paper_2609_07883_b200 import sharding as S
from paper_2609_07883_b200 import workloads as W


def test_shapes_and_slices_partition_the_heads():
    shape = W.AttnShape(16, 4, 64)
    assert S.shard_shape(shape, 2) == W.AttnShape(8, 2, 64)
    assert S.shard_shape(shape, 4) == W.AttnShape(4, 1, 64)
    with pytest.raises(ValueError):
        S.shard_shape(shape, 3)
    rng = np.random.default_rng(0)
    q = rng.integers(0, 1 << 16, size=(5, 16, 64)).astype(np.uint16)
    kv = rng.integers(0, 1 << 16, size=(5, 4, 64)).astype(np.uint16)
    pool = rng.integers(0, 1 << 16, size=7 * shape.page_elems).astype(np.uint16)
    for world in (1, 2, 4):
        assert np.array_equal(S.gather_heads([S.shard_rows(q, shape, r, world, "q") for r in range(world)]), q)
        assert np.array_equal(S.gather_heads([S.shard_rows(kv, shape, r, world, "kv") for r in range(world)]), kv)
        parts = [S.shard_pool(pool, shape, r, world).reshape(7, 2, 4 // world, 16, 64) for r in range(world)]
        assert np.array_equal(np.concatenate(parts, axis=2).reshape(-1), pool)
    # query head h reads KV head h // g: the q slice of a rank is exactly the heads that read its KV heads
    lo, hi = S.kv_head_range(shape, 1, 2)
    assert (lo, hi) == (2, 4) and S.shard_rows(q, shape, 1, 2, "q").shape[1] == (hi - lo) * shape.group
    assert np.array_equal(S.shard_rows(q, shape, 1, 2, "q"), q[:, lo * 4:hi * 4])


def test_sharded_oracle_equals_unsharded_oracle(oracle):
    """The definition itself: attention over a rank's heads on its slice of the pool equals those heads of the full
    result (bit for bit in the oracle, which computes head by head)."""
    rng = np.random.default_rng(3)
    shape = W.AttnShape(8, 4, 64)
    batch = W.make_batch(shape, 40, [5, 33, 100], 20, 37, rng)
    t = W.host_tensors(batch, rng)
    pool = t["pool"].copy()
    assert oracle.kv_append(pool, batch, t["k_new"], t["v_new"]) == 0
    full, full_lse, _ = oracle.mixed_attention(pool, batch, t["q"])
    full = full.reshape(batch.num_rows, shape.num_q_heads, shape.head_dim)
    full_lse = full_lse.reshape(batch.num_rows, shape.num_q_heads)
    for world in (2, 4):
        outs, lses = [], []
        for r in range(world):
            sb = S.shard_batch(batch, world)
            spool = S.shard_pool(t["pool"], shape, r, world).copy()
            assert oracle.kv_append(spool, sb, S.shard_rows(t["k_new"], shape, r, world, "kv"),
                                    S.shard_rows(t["v_new"], shape, r, world, "kv")) == 0
            assert np.array_equal(spool, S.shard_pool(pool, shape, r, world))
            o, l, _ = oracle.mixed_attention(spool, sb, S.shard_rows(t["q"], shape, r, world, "q"))
            outs.append(o.reshape(batch.num_rows, -1, shape.head_dim))
            lses.append(l.reshape(batch.num_rows, -1))
        assert np.array_equal(S.gather_heads(outs), full)
        assert np.array_equal(S.gather_heads(lses), full_lse)


def test_cost_tables_reduce_to_the_maximum_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "reduce.py"
    script.write_text(textwrap.dedent('''
        import json, os, sys
        import torch.distributed as dist
        sys.path.insert(0, os.environ["REPO"])
        from paper_2609_07883_b200 import sharding
        dist.init_process_group("gloo")
        r = dist.get_rank()
        tab = {"n_grid": [1, 2], "chunk_grid": [0, 16], "p50_ns": [[10 + r, 20 - r], [30, 40 + 5 * r]],
               "p99_ns": [[11 + 3 * r, 21], [31 - r, 41]]}
        out = sharding.reduce_table_max(tab)
        assert out["p50_ns"] == [[11, 20], [30, 45]], out
        assert out["p99_ns"] == [[14, 21], [31, 41]], out
        assert out["ranks_reduced"] == 2 and out["n_grid"] == [1, 2]
        dist.barrier()
        dist.destroy_process_group()
        print("rank", r, "ok")
    '''))
    env = dict(os.environ, REPO=os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)], env=env,
                         capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok") == 2


@pytest.mark.gpu
@pytest.mark.parametrize("world", [2, 4])
def test_ranks_side_by_side_equal_the_unsharded_launch(world, oracle):
    """Each rank's launch runs on this one GPU, one after the other (they are independent kernels); the outputs put side
    by side must equal the unsharded launch bit for bit, and the oracle within tolerance."""
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_07883_b200 import build

    build.build()
    from tests import gpu_util as G

    rng = np.random.default_rng(17)
    shape = W.AttnShape(16, 4, 128)
    batch = W.make_batch(shape, 400, [17, 256, 1000, 3000, 16], 64, 200, rng)
    t = W.host_tensors(batch, rng)
    full = G.Runner(batch, t)
    full.iterate()
    out_full, lse_full = full.results()
    assert full.status() == (0, 0)
    outs, lses, pools = [], [], []
    for r in range(world):
        sb = S.shard_batch(batch, world)
        st = {"pool": S.shard_pool(t["pool"], shape, r, world), "q": S.shard_rows(t["q"], shape, r, world, "q"),
              "k_new": S.shard_rows(t["k_new"], shape, r, world, "kv"), "v_new": S.shard_rows(t["v_new"], shape, r, world, "kv")}
        run = G.Runner(sb, st)
        run.iterate()
        o, l = run.results()
        assert run.status() == (0, 0)
        outs.append(o.reshape(batch.num_rows, -1, shape.head_dim))
        lses.append(l.reshape(batch.num_rows, -1))
        pools.append(G.torch_to_bits(run.pool).reshape(-1, 2, shape.num_kv_heads // world, 16, shape.head_dim))
    out_sharded = S.gather_heads(outs).reshape(out_full.shape)
    lse_sharded = S.gather_heads(lses).reshape(lse_full.shape)
    # the plan (split sizes) depends on the number of KV heads per rank, so sums may be reordered: tolerance, not bits
    pool_ref = t["pool"].copy()
    assert oracle.kv_append(pool_ref, batch, t["k_new"], t["v_new"]) == 0
    assert np.array_equal(np.concatenate(pools, axis=2).reshape(-1), pool_ref)
    ref, ref_lse, _ = oracle.mixed_attention(pool_ref, batch, t["q"])
    G.compare(out_sharded.reshape(-1, shape.head_dim), lse_sharded.reshape(-1), ref, ref_lse, f"sharded x{world}")
    assert np.abs(out_sharded - out_full).max() <= 2 * G.MAX_ABS

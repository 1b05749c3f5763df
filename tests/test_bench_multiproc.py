"""bench.py's N > 1 plumbing on CPU: two gloo ranks, max-over-ranks timing, whole-job aggregation, and the reference
arm's "rank 0 only" rule."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist

    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, str(ROOT))
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    per_rank_us = 100.0 + 50.0 * rank            # rank 1 is the slow one
    agg = bench.aggregate_result(per_rank_us, world, chunk=512, decodes=64)
    agg["sharded"] = bench.aggregate_result(per_rank_us, world, chunk=512, decodes=64, sharded=True)
    dist.barrier()
    Path(out_dir, f"rank{rank}.json").write_text(json.dumps(agg))
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_and_add_throughputs(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        agg = json.loads((tmp_path / f"rank{rank}.json").read_text())
        assert agg["value"] == 150.0                                   # the slowest rank decides
        assert abs(agg["iterations_per_s"] - 2 / 150e-6) < 1e-6        # two replicas finish one iteration each
        assert abs(agg["prefill_tokens_per_s"] - 2 * 512 / 150e-6) < 1e-3
        assert abs(agg["decode_tokens_per_s"] - 2 * 64 / 150e-6) < 1e-3
        # one iteration sharded by KV heads over the two ranks: still the slowest rank, but one iteration's tokens
        sh = agg["sharded"]
        assert sh["value"] == 150.0 and abs(sh["iterations_per_s"] - 1 / 150e-6) < 1e-6
        assert abs(sh["prefill_tokens_per_s"] - 512 / 150e-6) < 1e-3


def test_single_process_is_the_identity():
    sys.path.insert(0, str(ROOT))
    import bench

    assert bench.reduce_max_over_ranks(12.5) == 12.5


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "chat", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    r0 = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "chat", "--steps", "1",
                         "--warmup", "0", "--ref-seconds", "0.05"], env=env0, capture_output=True, text=True, timeout=300)
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "us" and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0

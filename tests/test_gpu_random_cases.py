"""Randomised parity: iterations whose shape, decode lengths, chunk list and launch form are drawn from a seed, compared
with the fp64 oracle on every output element (output, log-sum-exp) and on the whole pool after the append.

The draws favour the sizes where the kernels change behaviour: lengths of 1, 15-17, around 128 and 256 (page, KV tile
and unit edges), a few thousand tokens (requests cut into several units, work items cut into pieces), chunks of 1 to a
few hundred tokens at prefixes from 0 to several thousand, one to eight chunks, with and without decodes."""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W

pytestmark = pytest.mark.gpu

SHAPES = [W.AttnShape(8, 2, 128), W.TINY, W.AttnShape(4, 4, 64), W.AttnShape(8, 1, 128), W.AttnShape(4, 2, 128),
          W.AttnShape(16, 4, 64), W.AttnShape(16, 8, 128), W.AttnShape(16, 16, 64)]
EDGES = [1, 2, 15, 16, 17, 31, 33, 127, 128, 129, 255, 256, 257, 383, 511, 513]


@pytest.fixture(scope="module")
def gpu():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_07883_b200 import build

    build.build()
    from tests import gpu_util

    return gpu_util


def draw_length(rng, hi):
    """A length in [1, hi]: an edge value, a small one or a log-uniform one."""
    kind = rng.integers(0, 3)
    if kind == 0:
        return int(min(hi, EDGES[rng.integers(0, len(EDGES))]))
    if kind == 1:
        return int(rng.integers(1, min(hi, 300) + 1))
    return int(min(hi, np.exp(rng.uniform(0.0, np.log(hi)))) // 1) or 1


def draw_case(seed):
    """(shape, decode lengths, [(prefix, chunk tokens), ...], fused) for a seed."""
    rng = np.random.default_rng(90000 + seed)
    shape = SHAPES[rng.integers(0, len(SHAPES))]
    n = int(rng.choice([0, 1, 3, 7, 12]))
    lens = [draw_length(rng, 6000) for _ in range(n)]
    k = int(rng.choice([0, 1, 1, 1, 2, 3, 8])) if n else int(rng.choice([1, 1, 2, 5]))
    chunks = []
    for _ in range(k):
        prefix = 0 if rng.integers(0, 4) == 0 else draw_length(rng, 5000)
        chunks.append((int(prefix), draw_length(rng, 400)))
    return shape, lens, chunks, bool(rng.integers(0, 2))


def run_seed(gpu, oracle, seed):
    from tests.test_gpu_multichunk import oracle_rows

    shape, lens, chunks, fused = draw_case(seed)
    rng = np.random.default_rng(91000 + seed)
    pages = sum(-(-x // 16) for x in lens) + sum(-(-(p + c) // 16) for p, c in chunks) + 8
    what = f"seed {seed}: {shape}, decodes {lens}, chunks {chunks}, fused={fused}"
    if len(chunks) <= 1:
        P, C = chunks[0] if chunks else (0, 0)
        batch = W.make_batch(shape, pages, lens, P, C, rng)
    else:
        batch = W.make_multi_batch(shape, pages, lens, chunks, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    if fused:
        r.iterate()
    else:
        r.append()
        r.attend()
    out, lse = r.results()
    assert r.status() == (0, 0), f"{what}: device status {r.status()}"
    if len(chunks) <= 1:
        pool = t["pool"].copy()
        assert oracle.kv_append(pool, batch, t["k_new"], t["v_new"]) == 0
        ref, ref_lse, _ = oracle.mixed_attention(pool, batch, t["q"])
    else:
        pool, ref, ref_lse = oracle_rows(oracle, batch, t)
    assert np.array_equal(gpu.torch_to_bits(r.pool), pool), f"{what}: pool differs after append"
    d = shape.head_dim
    gpu.compare(out.reshape(-1, d), lse.reshape(-1), np.asarray(ref).reshape(-1, d), np.asarray(ref_lse).reshape(-1), what)


@pytest.mark.parametrize("seed", range(40))
def test_random_iteration_matches_the_oracle(gpu, oracle, seed):
    run_seed(gpu, oracle, seed)

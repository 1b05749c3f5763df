"""GPU parity of the chunk-prefill tensor-core tiles (and their mix with decode units) against the fp64 oracle."""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_07883_b200 import build

    build.build()
    from tests import gpu_util

    return gpu_util


def full_compare(gpu, oracle, batch, t, what):
    r = gpu.Runner(batch, t)
    r.append()
    r.attend()
    out, lse = r.results()
    assert r.status() == (0, 0), f"{what}: device status {r.status()}"
    pool = t["pool"].copy()
    assert oracle.kv_append(pool, batch, t["k_new"], t["v_new"]) == 0
    ref, ref_lse, _ = oracle.mixed_attention(pool, batch, t["q"])
    return gpu.compare(out.reshape(-1, batch.shape.head_dim), lse.reshape(-1), ref, ref_lse, what)


SHAPES = [W.AttnShape(8, 2, 128), W.TINY, W.AttnShape(4, 4, 64), W.AttnShape(8, 1, 128), W.AttnShape(4, 2, 128)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: f"{s.num_q_heads}q{s.num_kv_heads}kv{s.head_dim}d")
@pytest.mark.parametrize("P,C", [(0, 1), (0, 64), (37, 31), (128, 129), (300, 300), (1000, 257), (15, 513)])
def test_prefill_tiles_ragged(gpu, oracle, shape, P, C):
    rng = np.random.default_rng(1000 + P + C)
    batch = W.make_batch(shape, (P + C) // 16 + 8, [], P, C, rng)
    full_compare(gpu, oracle, batch, W.host_tensors(batch, rng), f"prefill P={P} C={C} {shape}")


@pytest.mark.parametrize("split", [[512], [128] * 4, [100, 412], [16] * 32, [257, 255]])
def test_chunk_invariance_on_gpu(gpu, oracle, split):
    """Any split of a prompt into chunks gives the rows of one unchunked causal prefill (within tolerance)."""
    rng = np.random.default_rng(77)
    shape = W.AttnShape(8, 2, 128)
    T = sum(split)
    q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
    k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    v = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    dense, dense_lse = oracle.dense_causal(q, k, v, shape.num_q_heads, shape.num_kv_heads, shape.head_dim)
    pages = np.random.default_rng(4).permutation(48)[: T // 16].astype(np.int32)
    first = W.MixedBatch(shape, 48, 0, split[0], pages[: -(-split[0] // 16)].copy(), np.zeros(0, np.int32),
                         np.zeros(1, np.int32), np.zeros(0, np.int32))
    tensors = {"pool": np.zeros(48 * shape.page_elems, np.uint16), "q": q[: split[0]], "k_new": k[: split[0]],
               "v_new": v[: split[0]]}
    r = gpu.Runner(first, tensors)
    B = r.B
    import torch

    P = 0
    got, got_lse = [], []
    for c in split:
        b = W.MixedBatch(shape, 48, P, c, pages[: -(-(P + c) // 16)].copy(), np.zeros(0, np.int32), np.zeros(1, np.int32),
                         np.zeros(0, np.int32))
        ctx = B.Context(shape, 48, c, 1, 64)
        db = B.DeviceBatch(b, r.dev)
        qd, kd, vd = (gpu.bits_to_torch(x[P:P + c], r.dev) for x in (q, k, v))
        od = torch.zeros_like(qd)
        ld = torch.zeros(c, shape.num_q_heads, dtype=torch.float32, device=r.dev)
        B.sw_kv_append(ctx, r.pool, db, kd, vd)
        B.sw_mixed_attn_run(ctx, r.pool, db, qd, od, ld)
        torch.cuda.synchronize()
        assert B.sw_check_status(ctx, raise_on_error=False) == (0, 0)
        got.append(W.bf16_bits_to_f64(gpu.torch_to_bits(od)))
        got_lse.append(ld.cpu().numpy().astype(np.float64))
        P += c
    gpu.compare(np.concatenate(got).reshape(-1, 128), np.concatenate(got_lse).reshape(-1), dense.reshape(-1, 128),
                dense_lse.reshape(-1), f"split {split}")


def test_mixed_iteration_with_long_prefix_and_decodes(gpu, oracle):
    rng = np.random.default_rng(78)
    shape = W.AttnShape(8, 2, 128)
    lens = [700, 33, 2049, 5000]
    P, C = 2000, 200
    need = sum(-(-x // 16) for x in lens) + (P + C) // 16 + 4
    batch = W.make_batch(shape, need, lens, P, C, rng)
    full_compare(gpu, oracle, batch, W.host_tensors(batch, rng), "mixed long prefix")


def test_constant_v_and_causal_closed_forms(gpu, oracle):
    import torch

    rng = np.random.default_rng(79)
    shape = W.AttnShape(8, 2, 128)
    T = 300
    batch = W.make_batch(shape, 32, [], 0, T, rng)
    # V == 1 -> output == 1 exactly representable; K random
    t = W.host_tensors(batch, rng)
    t["pool"][:] = 0
    t["v_new"] = W.f32_to_bf16_bits(np.ones((T, 2, 128), np.float32))
    r = gpu.Runner(batch, t)
    r.append()
    r.attend()
    out, _ = r.results()
    assert np.max(np.abs(out - 1.0)) <= 2 ** -7
    # causal inclusivity closed form: K == 0, V[t][0] = t/256 -> row p gives p/512 (positions <= 256 exact in bf16)
    t2 = W.host_tensors(batch, rng)
    t2["pool"][:] = 0
    t2["k_new"][:] = 0
    vf = np.zeros((T, 2, 128), np.float32)
    vf[:, :, 0] = (np.arange(T, dtype=np.float32) / 256.0)[:, None]
    t2["v_new"] = W.f32_to_bf16_bits(vf)
    r2 = gpu.Runner(batch, t2)
    r2.append()
    r2.attend()
    out2, _ = r2.results()
    p = np.arange(257, dtype=np.float64)
    for h in range(8):
        assert np.max(np.abs(out2[:257, h, 0] - p / 512.0)) <= 4e-3


@pytest.mark.parametrize("P,C", [(6000, 64), (20000, 32), (12000, 200)])
def test_long_prefix_small_chunk_is_cut_into_pieces_and_merged(gpu, oracle, P, C):
    """Few items with many KV tiles: each item is cut along the KV axis, published as partials and merged."""
    rng = np.random.default_rng(P + C)
    shape = W.AttnShape(8, 2, 128)
    batch = W.make_batch(shape, (P + C) // 16 + 40, [300, 5], P, C, rng)
    full_compare(gpu, oracle, batch, W.host_tensors(batch, rng), f"pieces P={P} C={C}")

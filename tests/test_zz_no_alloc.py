"""The non-allocating entry point (sw_decode_attn_static) against the ordinary one.

Some callers of this library may not allocate device memory — a plugin living inside another runtime's memory pool,
or a latency-critical loop where cudaMalloc would stall the device — so they can create neither a context nor a
workspace.  For them the library keeps the decode kernel's scratch in a fixed array inside its own image.  This
test calls that entry point through the C-ABI twice in a row (the array keeps the previous call's contents, so the
second call proves that it is cleared where it must be) and compares with sw_mixed_attn_run on the same inputs.
It is collected last so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_context_entry_point(oracle):
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_07883_b200 import build

    build.build()
    from paper_2609_07883_b200 import binding as B
    from tests import gpu_util as G

    rng = np.random.default_rng(4242)
    shape = W.AttnShape(8, 2, 128)
    lens = [1, 17, 300, 2500, 9000, 64]          # the long ones are split and merged through the static scratch
    need = sum(-(-x // 16) for x in lens)
    batch = W.make_batch(shape, need + 8, lens, 0, 0, rng)
    t = W.host_tensors(batch, rng)
    r = G.Runner(batch, t)
    r.append()
    r.attend()                                    # the existing entry point (context + caller's workspace)
    want, want_lse = r.results()
    layout = B.make_layout(shape, batch.num_pages)
    for call in range(2):
        out = torch.zeros_like(r.q)
        lse = torch.zeros_like(r.lse)
        B.sw_decode_attn_static(layout, 0, r.pool, r.dbatch, r.q, out, lse)
        torch.cuda.synchronize()
        got = W.bf16_bits_to_f64(G.torch_to_bits(out))
        G.compare(got.reshape(-1, 128), lse.cpu().numpy().astype(np.float64).reshape(-1), want.reshape(-1, 128),
                  want_lse.reshape(-1), f"static scratch, call {call}")
    # and against the oracle, like every other parity test
    ref, ref_lse, _ = oracle.mixed_attention(G.torch_to_bits(r.pool), batch, t["q"])
    G.compare(got.reshape(-1, 128), lse.cpu().numpy().astype(np.float64).reshape(-1), ref, ref_lse, "static scratch vs oracle")
    # sizes beyond the stated maximum are refused with a clear error, nothing is launched
    big = W.make_batch(shape, 4 * (B.SW_STATIC_MAX_DECODE + 1) + 8, [20] * (B.SW_STATIC_MAX_DECODE + 1), 0, 0, rng)
    with pytest.raises(B.SwError) as e:
        B.sw_decode_attn_static(B.make_layout(shape, big.num_pages), 0, r.pool, B.DeviceBatch(big, r.dev), r.q, out)
    assert e.value.status == B.SW_ERR_WORKSPACE and "static limit" in str(e.value)
    chunked = W.make_batch(shape, 64, [20], 0, 16, rng)
    with pytest.raises(B.SwError) as e:
        B.sw_decode_attn_static(B.make_layout(shape, 64), 0, r.pool, B.DeviceBatch(chunked, r.dev), r.q, out)
    assert e.value.status == B.SW_ERR_UNSUPPORTED


@pytest.mark.parametrize("shape,lens", [
    # exactly the stated maximum of requests with 8 KV heads: every ticket / ready slot of the fixed array is in use and
    # the unit count comes close to the array's partial-result slots (a few contexts of thousands of tokens among
    # one-page ones)
    (W.AttnShape(32, 8, 128), [16] * 100 + [1, 15, 17, 33] * 5 + [6000, 9000, 12000, 20000, 2500, 3100, 700, 129]),
    # head size 64 with eight query heads per KV head, and one query head per KV head
    (W.AttnShape(8, 1, 64), [5000, 40, 16, 2100, 333]),
    (W.AttnShape(4, 4, 64), [3000, 1, 200]),
], ids=["max_requests_8kv", "d64_group8", "d64_group1"])
def test_static_scratch_at_its_limits(oracle, shape, lens):
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_07883_b200 import build

    build.build()
    from paper_2609_07883_b200 import binding as B
    from tests import gpu_util as G

    if shape.num_kv_heads == 8:
        assert len(lens) == B.SW_STATIC_MAX_DECODE
    rng = np.random.default_rng(4243)
    batch = W.make_batch(shape, sum(-(-x // 16) for x in lens) + 8, lens, 0, 0, rng)
    t = W.host_tensors(batch, rng)
    r = G.Runner(batch, t)
    r.append()
    r.attend()
    want, want_lse = r.results()
    ref, ref_lse, _ = oracle.mixed_attention(G.torch_to_bits(r.pool), batch, t["q"])
    layout = B.make_layout(shape, batch.num_pages)
    d = shape.head_dim
    for call in range(2):
        out = torch.zeros_like(r.q)
        lse = torch.zeros_like(r.lse)
        B.sw_decode_attn_static(layout, 0, r.pool, r.dbatch, r.q, out, lse)
        torch.cuda.synchronize()
        got = W.bf16_bits_to_f64(G.torch_to_bits(out)).reshape(-1, d)
        got_lse = lse.cpu().numpy().astype(np.float64).reshape(-1)
        G.compare(got, got_lse, want.reshape(-1, d), want_lse.reshape(-1), f"static scratch at its limits, call {call}")
        G.compare(got, got_lse, ref, ref_lse, f"static scratch at its limits vs oracle, call {call}")

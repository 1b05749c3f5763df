"""GPU parity: the CUDA path, called through the C-ABI, against the fp64 oracle on the same seeded inputs."""
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


def run_and_compare(gpu, oracle, batch, tensors, pairs=None, what="", fused=False):
    r = gpu.Runner(batch, tensors)
    if fused:
        r.iterate()
    else:
        r.append()
        r.attend()
    out, lse = r.results()
    assert r.status() == (0, 0), f"{what}: device status {r.status()}"
    # oracle on its own copy of the pool, appended by the oracle
    pool = tensors["pool"].copy()
    assert oracle.kv_append(pool, batch, tensors["k_new"], tensors["v_new"]) == 0
    assert np.array_equal(gpu.torch_to_bits(r.pool), pool), f"{what}: pool differs after append"
    sh = batch.shape
    if pairs is None:
        ref, ref_lse, _ = oracle.mixed_attention(pool, batch, tensors["q"])
        g = out.reshape(-1, sh.head_dim)
        gl = lse.reshape(-1)
    else:
        pairs = np.asarray(pairs, dtype=np.int32)
        ref, ref_lse, _ = oracle.mixed_attention(pool, batch, tensors["q"], pairs=pairs)
        g = out[pairs[:, 0], pairs[:, 1]]
        gl = lse[pairs[:, 0], pairs[:, 1]]
    return gpu.compare(g, gl, ref, ref_lse, what)


def test_tiny_workload_full(gpu, oracle):
    rng = W.rng_for(0)
    batch = W.tiny_batch(rng)
    t = W.host_tensors(batch, rng)
    run_and_compare(gpu, oracle, batch, t, what="tiny")


@pytest.mark.parametrize("shape", [W.TINY, W.AttnShape(8, 2, 128), W.AttnShape(4, 4, 64), W.AttnShape(8, 1, 128),
                                   W.AttnShape(4, 2, 128)])
def test_ragged_small_cases(gpu, oracle, shape):
    rng = np.random.default_rng(31)
    lens = [1, 15, 16, 17, 31, 255, 256, 257, 700]
    batch = W.make_batch(shape, 160, lens, 37, 91, rng)
    t = W.host_tensors(batch, rng)
    run_and_compare(gpu, oracle, batch, t, what=f"ragged {shape}")


@pytest.mark.parametrize("case", ["tiny", "ragged", "ragged_d64", "decode_only", "prefill_only", "long_split", "chat"])
def test_fused_iteration_matches_oracle(gpu, oracle, case):
    """Append and attention in one launch: the rows written at the start of the kernel are the ones the diagonal tiles
    and every request's last page must see."""
    rng = np.random.default_rng(77)
    pairs = None
    if case == "tiny":
        batch = W.tiny_batch(rng)
    elif case == "ragged":
        batch = W.make_batch(W.AttnShape(8, 2, 128), 200, [1, 15, 16, 17, 31, 255, 256, 257, 700], 37, 91, rng)
    elif case == "ragged_d64":
        batch = W.make_batch(W.AttnShape(4, 4, 64), 200, [1, 16, 17, 333, 700], 128, 300, rng)
    elif case == "decode_only":
        batch = W.make_batch(W.TINY, 120, [5, 64, 300, 301, 1], 0, 0, rng)
    elif case == "prefill_only":
        batch = W.make_batch(W.TINY, 120, [], 200, 333, rng)
    elif case == "long_split":
        batch = W.make_batch(W.AttnShape(8, 2, 128), 1400, [20000, 3], 0, 0, rng)
    else:
        batch = W.chat_batch(n=64, chunk_len=512, prefix_len=512, rng=rng)
        rows = rng.choice(batch.num_rows, size=96, replace=False)
        pairs = [(int(r), int(rng.integers(batch.shape.num_q_heads))) for r in rows]
        pairs += [(batch.chunk_len - 1, 0), (batch.chunk_len, 1), (batch.num_rows - 1, 2)]
    t = W.host_tensors(batch, rng)
    run_and_compare(gpu, oracle, batch, t, pairs=pairs, what=f"fused {case}", fused=True)


def test_fused_iteration_repeated_with_new_rows(gpu, oracle):
    """Several fused launches in a row on one context, each appending different rows at the same positions: a launch
    that read a page before its rows were written would return the previous launch's values."""
    rng = np.random.default_rng(78)
    batch = W.make_batch(W.AttnShape(8, 2, 128), 400, [17, 256, 1000, 4000, 16], 64, 200, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    for it in range(4):
        t["k_new"] = W.normal_bf16_bits(rng, *t["k_new"].shape)
        t["v_new"] = W.normal_bf16_bits(rng, *t["v_new"].shape)
        r.k_new = gpu.bits_to_torch(t["k_new"], r.dev)
        r.v_new = gpu.bits_to_torch(t["v_new"], r.dev)
        r.iterate()
        out, lse = r.results()
        assert r.status() == (0, 0)
        pool = t["pool"]
        assert oracle.kv_append(pool, batch, t["k_new"], t["v_new"]) == 0
        assert np.array_equal(gpu.torch_to_bits(r.pool), pool), f"launch {it}: pool differs after append"
        ref, ref_lse, _ = oracle.mixed_attention(pool, batch, t["q"])
        gpu.compare(out.reshape(-1, batch.shape.head_dim), lse.reshape(-1), ref, ref_lse, f"fused launch {it}")


def test_decode_only_and_prefill_only(gpu, oracle):
    rng = np.random.default_rng(32)
    b1 = W.make_batch(W.TINY, 64, [5, 300, 77], 0, 0, rng)
    run_and_compare(gpu, oracle, b1, W.host_tensors(b1, rng), what="decode-only")
    b2 = W.make_batch(W.TINY, 64, [], 130, 70, rng)
    run_and_compare(gpu, oracle, b2, W.host_tensors(b2, rng), what="prefill-only")
    b3 = W.make_batch(W.TINY, 64, [], 0, 33, rng)
    run_and_compare(gpu, oracle, b3, W.host_tensors(b3, rng), what="prefill at P=0")


def test_long_decode_is_split_and_merged(gpu, oracle):
    """Contexts far above the minimum split length exercise the split-KV units and the last-arriver merge."""
    rng = np.random.default_rng(33)
    lens = [9000, 4097, 12345, 300]
    need = sum(-(-x // 16) for x in lens)
    batch = W.make_batch(W.AttnShape(8, 2, 128), need + 8, lens, 0, 0, rng)
    t = W.host_tensors(batch, rng)
    run_and_compare(gpu, oracle, batch, t, what="split decode")
    # twice in a row on one context: tickets and counters must re-arm themselves
    r = gpu.Runner(batch, t)
    r.append()
    r.attend()
    first, _ = r.results()
    r.out.zero_()
    r.attend()
    second, _ = r.results()
    assert np.array_equal(first, second)


def test_length_one_rows_return_v0_bit_exactly(gpu, oracle):
    rng = np.random.default_rng(34)
    batch = W.make_batch(W.TINY, 32, [1, 1, 40], 0, 3, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    r.append()
    r.attend()
    out_bits = gpu.torch_to_bits(r.out)
    g = batch.shape.group
    for h in range(batch.shape.num_q_heads):
        assert np.array_equal(out_bits[0, h], t["v_new"][0, h // g])      # chunk row 0 at P = 0
        assert np.array_equal(out_bits[3, h], t["v_new"][3, h // g])      # decode with one key
        assert np.array_equal(out_bits[4, h], t["v_new"][4, h // g])


def test_nan_in_unwritten_slots_of_the_last_page_does_not_leak(gpu, oracle):
    rng = np.random.default_rng(35)
    batch = W.make_batch(W.AttnShape(8, 2, 128), 64, [5, 33, 250], 20, 45, rng)
    t = W.host_tensors(batch, rng)
    t["pool"][:] = 0x7FC0  # every slot NaN until written
    # fill the already-cached positions (prefix and earlier decode tokens) with finite values
    pool = t["pool"]
    pv = pool.reshape(batch.num_pages, 2, 2, 16, 128)
    S = 16
    for pos in range(batch.prefix_len):
        pv[batch.prefill_pages[pos // S], :, :, pos % S, :] = W.normal_bf16_bits(rng, 2, 2, 128)
    for i, L in enumerate(batch.decode_kv_len):
        pages = batch.decode_pages[batch.decode_page_indptr[i]:]
        for pos in range(int(L) - 1):
            pv[pages[pos // S], :, :, pos % S, :] = W.normal_bf16_bits(rng, 2, 2, 128)
    run_and_compare(gpu, oracle, batch, t, what="NaN tail")


def test_page_permutation_invariance(gpu, oracle):
    rng = np.random.default_rng(36)
    shape = W.AttnShape(8, 2, 128)
    outs = []
    for seed in (1, 2):
        batch = W.make_batch(shape, 96, [100, 333], 50, 60, np.random.default_rng(seed))
        trng = np.random.default_rng(99)
        t = W.host_tensors(batch, trng, with_pool=False)
        t["pool"] = np.zeros(batch.num_pages * shape.page_elems, np.uint16)
        # write the cached history through the oracle-independent append of the CUDA path itself: first an
        # iteration that appends the history, then the iteration under test
        hist = W.MixedBatch(shape, batch.num_pages, 0, 50, batch.prefill_pages[:4].copy(), np.zeros(0, np.int32),
                            np.zeros(1, np.int32), np.zeros(0, np.int32))
        hk = W.normal_bf16_bits(np.random.default_rng(7), 50, 2, 128)
        hv = W.normal_bf16_bits(np.random.default_rng(8), 50, 2, 128)
        assert oracle.kv_append(t["pool"], hist, hk, hv) == 0
        for i, L in enumerate(batch.decode_kv_len):
            one = W.MixedBatch(shape, batch.num_pages, 0, int(L) - 1,
                               batch.decode_pages[batch.decode_page_indptr[i]:batch.decode_page_indptr[i + 1]].copy(),
                               np.zeros(0, np.int32), np.zeros(1, np.int32), np.zeros(0, np.int32))
            dk = W.normal_bf16_bits(np.random.default_rng(10 + i), int(L) - 1, 2, 128)
            dv = W.normal_bf16_bits(np.random.default_rng(20 + i), int(L) - 1, 2, 128)
            assert oracle.kv_append(t["pool"], one, dk, dv) == 0
        r = gpu.Runner(batch, t)
        r.append()
        r.attend()
        outs.append(gpu.torch_to_bits(r.out).copy())
        run_and_compare(gpu, oracle, batch, t, what=f"perm {seed}")
    assert np.array_equal(outs[0], outs[1])


def test_bad_page_ids_are_reported_not_faulted(gpu, oracle):
    rng = np.random.default_rng(37)
    batch = W.make_batch(W.TINY, 64, [40, 70], 10, 20, rng)
    t = W.host_tensors(batch, rng)
    bad = W.MixedBatch(**{**batch.__dict__})
    bad.decode_pages = batch.decode_pages.copy()
    bad.decode_pages[1] = batch.num_pages + 5
    r = gpu.Runner(bad, t)
    r.attend()
    code, detail = r.status()
    assert code == r.B.SW_ERR_OUT_OF_RANGE
    assert r.status() == (0, 0)           # cleared by the read
    bad2 = W.MixedBatch(**{**batch.__dict__})
    bad2.prefill_pages = batch.prefill_pages.copy()
    bad2.prefill_pages[-1] = -3
    r2 = gpu.Runner(bad2, t)
    r2.append()
    assert r2.status()[0] == r2.B.SW_ERR_OUT_OF_RANGE
    # the same bad prompt page id in the attention call: the chunk-prefill producer reports it and reads page 0 in its
    # place (no out-of-range coordinate reaches the copy engine); likewise for ids whose doubled value would wrap
    for bad_id in (-3, batch.num_pages, (1 << 30) + 1, -(1 << 30) - 7):
        bad3 = W.MixedBatch(**{**batch.__dict__})
        bad3.prefill_pages = batch.prefill_pages.copy()
        bad3.prefill_pages[0] = bad_id
        r3 = gpu.Runner(bad3, t)
        r3.attend()
        assert r3.status()[0] == r3.B.SW_ERR_OUT_OF_RANGE, bad_id
        assert r3.status() == (0, 0)
        bad4 = W.MixedBatch(**{**batch.__dict__})
        bad4.decode_pages = batch.decode_pages.copy()
        bad4.decode_pages[0] = bad_id
        r4 = gpu.Runner(bad4, t)
        r4.attend()
        assert r4.status()[0] == r4.B.SW_ERR_OUT_OF_RANGE, bad_id
    # a good iteration on the same context still works afterwards
    run_and_compare(gpu, oracle, batch, t, what="after bad ids")


def test_calls_refuse_a_context_of_another_device(gpu):
    """A context serves the device it was created on: with another device named or current the launching calls return
    SW_ERR_INVALID_ARG and launch nothing.  (One GPU is enough: the static entry point is told a device that is not
    the current one.)"""
    import torch

    from paper_2609_07883_b200 import binding as B

    rng = np.random.default_rng(41)
    batch = W.make_batch(W.TINY, 64, [40], 0, 0, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    with pytest.raises(B.SwError) as e:
        B.sw_decode_attn_static(B.make_layout(W.TINY, 64), 1, r.pool, r.dbatch, r.q, r.out)
    assert e.value.status == B.SW_ERR_INVALID_ARG and "is current" in str(e.value)
    if torch.cuda.device_count() > 1:
        with torch.cuda.device(1):
            with pytest.raises(B.SwError) as e:
                B.sw_mixed_attn_run(r.ctx, r.pool, r.dbatch, r.q, r.out)
            assert e.value.status == B.SW_ERR_INVALID_ARG and "is current" in str(e.value)
    # creating a context leaves the caller's current device as it was
    assert torch.cuda.current_device() == 0


def test_host_argument_errors(gpu):
    from paper_2609_07883_b200 import binding as B

    rng = np.random.default_rng(38)
    batch = W.make_batch(W.TINY, 64, [40], 10, 20, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    short = W.MixedBatch(**{**batch.__dict__})
    short.prefill_pages = batch.prefill_pages[:-1].copy()
    db = B.DeviceBatch(short, r.dev)
    with pytest.raises(B.SwError) as e:
        B.sw_mixed_attn_run(r.ctx, r.pool, db, r.q, r.out)
    assert e.value.status == B.SW_ERR_OUT_OF_RANGE
    big = W.make_batch(W.TINY, 64, [40], 10, 40, rng)   # chunk beyond the context's max_chunk
    with pytest.raises(B.SwError) as e:
        B.sw_mixed_attn_run(r.ctx, r.pool, B.DeviceBatch(big, r.dev), r.q, r.out)
    assert e.value.status == B.SW_ERR_WORKSPACE
    # q and out are read and written through tensor maps: a pointer off the 16-byte grid is refused, nothing is launched
    import torch

    wide = torch.zeros(r.out.numel() + 8, dtype=r.out.dtype, device=r.out.device)
    skewed = wide[1:1 + r.out.numel()].view(r.out.shape)   # 2 bytes past an aligned address
    for q, out in ((r.q, skewed), (skewed, r.out)):
        with pytest.raises(B.SwError) as e:
            B.sw_mixed_attn_run(r.ctx, r.pool, r.dbatch, q, out)
        assert e.value.status == B.SW_ERR_INVALID_ARG and "16-byte aligned" in str(e.value)
    assert B.sw_check_status(r.ctx, raise_on_error=False) == (0, 0)


def test_host_buffer_iteration_matches_device_path(gpu, oracle):
    import torch

    rng = np.random.default_rng(39)
    batch = W.make_batch(W.AttnShape(8, 2, 128), 96, [100, 333, 17], 50, 60, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    B = r.B
    hs, keep = B.host_batch_struct(batch)
    h_out = np.zeros_like(t["q"])
    h_lse = np.zeros((batch.num_rows, batch.shape.num_q_heads), np.float32)
    B.sw_mixed_iteration_host(r.ctx, r.pool, hs, t["q"], t["k_new"], t["v_new"], h_out, h_lse)
    pool = t["pool"].copy()
    oracle.kv_append(pool, batch, t["k_new"], t["v_new"])
    assert np.array_equal(gpu.torch_to_bits(r.pool), pool)
    ref, ref_lse, _ = oracle.mixed_attention(pool, batch, t["q"])
    gpu.compare(W.bf16_bits_to_f64(h_out).reshape(-1, 128), h_lse.reshape(-1).astype(np.float64), ref, ref_lse, "host path")


def test_chat_workload_sampled_rows(gpu, oracle):
    rng = W.rng_for(1)
    batch = W.chat_batch(n=16, chunk_len=128, rng=rng)
    t = W.host_tensors(batch, rng)
    C, n, Hq = batch.chunk_len, batch.num_decode, batch.shape.num_q_heads
    rows = [0, 1, 15, 16, 17, 31, 32, 63, 64, 127] + [C + i for i in range(n)]
    prs = np.random.default_rng(5)
    pairs = [(r_, int(prs.integers(0, Hq))) for r_ in rows] + [(r_, int(prs.integers(0, Hq))) for r_ in rows]
    run_and_compare(gpu, oracle, batch, t, pairs=pairs, what="chat n=16 C=128")


def test_many_decode_requests(gpu, oracle):
    """1500 requests: the in-kernel plan scans several requests per thread and the unit search spans the whole list."""
    rng = np.random.default_rng(40)
    lens = rng.integers(1, 90, size=1500)
    need = int(sum(-(-int(x) // 16) for x in lens)) + 8
    batch = W.make_batch(W.TINY, need, lens, 0, 0, rng)
    run_and_compare(gpu, oracle, batch, W.host_tensors(batch, rng), what="n=1500")


def test_short_page_list_is_reported_and_the_context_recovers(gpu, oracle):
    """A request whose page list is shorter than its length: its units are skipped and reported; reading the status
    re-arms the context, and the next (good) iteration on the same context is correct."""
    rng = np.random.default_rng(41)
    shape = W.AttnShape(8, 2, 128)
    lens = [5000, 3000]
    need = sum(-(-x // 16) for x in lens) + 8
    batch = W.make_batch(shape, need, lens, 0, 0, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    B = r.B
    bad = W.MixedBatch(**{**batch.__dict__})
    bad.decode_page_indptr = batch.decode_page_indptr.copy()
    bad.decode_page_indptr[1:] -= 100          # request 0 now owns 100 pages fewer than 5000 tokens need
    bad.decode_pages = np.concatenate([batch.decode_pages[:batch.decode_page_indptr[1] - 100],
                                       batch.decode_pages[batch.decode_page_indptr[1]:]])
    B.sw_mixed_attn_run(r.ctx, r.pool, B.DeviceBatch(bad, r.dev), r.q, r.out)
    code, _ = r.status()
    assert code == B.SW_ERR_OUT_OF_RANGE
    r.append()
    r.attend()
    out, lse = r.results()
    assert r.status() == (0, 0)
    pool = t["pool"].copy()
    oracle.kv_append(pool, batch, t["k_new"], t["v_new"])
    ref, ref_lse, _ = oracle.mixed_attention(pool, batch, t["q"])
    gpu.compare(out.reshape(-1, 128), lse.reshape(-1), ref, ref_lse, "after recovery")


def test_a_wait_that_cannot_succeed_gives_up_and_the_context_stays_usable(gpu, oracle):
    """Failure detection without a fault: a bounded wait runs out (nothing ever completes its barrier), the kernel ends
    normally with SW_ERR_DEVICE_TIMEOUT in the status word, and the same context then runs a correct iteration."""
    import time

    rng = np.random.default_rng(42)
    batch = W.make_batch(W.TINY, 64, [40, 70], 10, 20, rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    t0 = time.time()
    r.B.sw_selftest_wait_timeout(r.ctx, 200_000)          # about 0.1 ms of SM clock
    code, detail = r.status()
    assert time.time() - t0 < 5.0
    assert code == r.B.SW_ERR_DEVICE_TIMEOUT and (detail & 0xFFFFFF) == 0xABCD
    assert r.status() == (0, 0)
    run_and_compare(gpu, oracle, batch, t, what="after a timed-out wait")


@pytest.mark.parametrize("heads", [(8, 1, 128), (8, 2, 128), (4, 2, 64), (8, 8, 64)])
def test_many_splits_of_one_request_share_the_merge(gpu, oracle, heads):
    """One long context beside a short one is cut into dozens of units per KV head; from a few dozen splits on, the
    units that draw the last tickets merge one row of the group each (group sizes 8, 4, 2; group 1 keeps the single
    merger).  Run twice: the shared counters must re-arm themselves."""
    rng = np.random.default_rng(35)
    lens = [20011, 500]
    need = sum(-(-x // 16) for x in lens)
    batch = W.make_batch(W.AttnShape(*heads), need + 8, lens, 0, 0, rng)
    t = W.host_tensors(batch, rng)
    run_and_compare(gpu, oracle, batch, t, what=f"wide merge {heads}")
    r = gpu.Runner(batch, t)
    r.append()
    r.attend()
    first, _ = r.results()
    r.out.zero_()
    r.attend()
    second, _ = r.results()
    assert r.status() == (0, 0)
    assert np.array_equal(first, second)


def test_many_long_requests_in_several_rounds(gpu, oracle):
    """Six 30k-token requests over 8 KV heads: more pages than one round of units can take, so warps run several units
    and pull them from the counter, and every request has dozens of units whose merge is shared by fixed mergers that
    claim their next unit late.  Twice in a row: the counters must re-arm themselves."""
    rng = np.random.default_rng(36)
    shape = W.AttnShape(16, 8, 64)
    lens = [30000 + 37 * i for i in range(6)]
    need = sum(-(-x // 16) for x in lens)
    batch = W.make_batch(shape, need + 8, lens, 0, 0, rng)
    t = W.host_tensors(batch, rng)
    run_and_compare(gpu, oracle, batch, t, what="several rounds of units, shared merges")
    r = gpu.Runner(batch, t)
    r.append()
    r.attend()
    first, _ = r.results()
    r.out.zero_()
    r.attend()
    second, _ = r.results()
    assert r.status() == (0, 0)
    assert np.array_equal(first, second)

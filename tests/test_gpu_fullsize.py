"""Full-size parity: the workloads bench.py times (and the larger ones), in the same launch configuration, checked on
sampled outputs that the oracle computes one by one; the KV pools after append are compared whole, bit for bit."""
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


def run_case(gpu, oracle, batch, pairs, seed, what, **kw):
    return gpu.run_device_case(oracle, batch, pairs, seed, what, **kw)


def sample_pairs(batch, rng, chunk_rows, n_decode_extra):
    C, n, Hq = batch.chunk_len, batch.num_decode, batch.shape.num_q_heads
    rows = [r for r in chunk_rows if 0 <= r < C]
    if n:
        lens = batch.decode_kv_len
        rows += [C + int(np.argmin(lens)), C + int(np.argmax(lens))]
        rows += [C + int(i) for i in rng.choice(n, size=min(n, n_decode_extra), replace=False)]
    return [(r, int(rng.integers(0, Hq))) for r in rows]


def test_chat_workload_as_benchmarked(gpu, oracle):
    rng = W.rng_for(1)
    batch = W.chat_batch(n=64, chunk_len=512, prefix_len=512, rng=rng)
    pairs = sample_pairs(batch, np.random.default_rng(1), [0, 1, 15, 16, 31, 32, 63, 64, 127, 128, 255, 256, 383, 511], 12)
    run_case(gpu, oracle, batch, pairs, 101, "chat n=64 C=512 P=512")


def test_mixed_workload_cost_surface_point(gpu, oracle):
    rng = W.rng_for(2)
    batch = W.mixed_batch(1024, 4096, n=128, rng=rng)
    pairs = sample_pairs(batch, np.random.default_rng(2), [0, 31, 32, 127, 128, 129, 511, 512, 1000, 1023], 16)
    run_case(gpu, oracle, batch, pairs, 102, "mixed n=128 C=1024 P=4096")


@pytest.mark.parametrize("C,P", [(256, 28672), (512, 16384), (64, 28672)])
def test_fewer_items_than_sms_beside_many_decode_pages(gpu, oracle, C, P):
    """32, 64 or 8 work items of 130 to 225 KV tiles beside the 128 log-normal decodes (1.4 GB of pages): the number of
    pieces per item is the one that ends the launch soonest when the SMs without a piece stream decode pages meanwhile."""
    batch = W.mixed_batch(C, P, n=128, rng=W.rng_for(2))
    pairs = sample_pairs(batch, np.random.default_rng(12), gpu.boundary_rows(C, batch.shape.group), 16)
    run_case(gpu, oracle, batch, pairs, 160 + C, f"mixed n=128 C={C} P={P}", fused=True)


def test_long_context_workload(gpu, oracle):
    rng = W.rng_for(3)
    batch = W.long_batch(1024, 98304, n=16, rng=rng)
    pairs = sample_pairs(batch, np.random.default_rng(3), [0, 1, 63, 64, 512, 1023], 6)
    run_case(gpu, oracle, batch, pairs, 103, "long n=16 C=1024 P=98304")


def edge_pairs(gpu, batch, rng, n_decode_extra):
    """(row, head) sample of a large case: the chunk rows next to every tile, KV-tile and (sampled) page edge, the
    shortest and the longest decode and a few more, one random query head each."""
    return sample_pairs(batch, rng, gpu.boundary_rows(batch.chunk_len, batch.shape.group), n_decode_extra)


@pytest.mark.parametrize("C", [2048, 4096])
def test_prefill_only_large_chunk_at_prefix_zero(gpu, oracle, C):
    """The chunk sizes the tensor-core target is stated on, at prefix 0: 256 / 512 work items of 1 to 32 KV tiles, pulled
    longest first from the counter over several waves."""
    batch = W.make_batch(W.LLAMA, C // 16 + 64, [], 0, C, np.random.default_rng(40 + C))
    run_case(gpu, oracle, batch, edge_pairs(gpu, batch, np.random.default_rng(5), 0), 140 + C, f"prefill-only C={C} P=0")


def test_mixed_workload_large_chunk_fused(gpu, oracle):
    """C=4096 at prefix 28672 beside the 128 log-normal decodes, append and attention in one launch."""
    batch = W.mixed_batch(4096, 28672, n=128, rng=W.rng_for(2))
    run_case(gpu, oracle, batch, edge_pairs(gpu, batch, np.random.default_rng(6), 16), 104,
             "mixed n=128 C=4096 P=28672 (fused)", fused=True)


def test_long_context_workload_large_chunks(gpu, oracle):
    """C=8192 and C=4096 at prefix 98304 beside the 16 decodes of 32k-131k tokens (the largest single-GPU configuration,
    and the one bench.py times by default): 1024 / 512 work items of about 800 KV tiles each."""
    import dataclasses

    big = W.long_batch(8192, 98304, n=16, rng=W.rng_for(3))
    run_case(gpu, oracle, big, edge_pairs(gpu, big, np.random.default_rng(7), 4), 105, "long n=16 C=8192 P=98304", fused=True)
    half = dataclasses.replace(big, chunk_len=4096)
    run_case(gpu, oracle, half, edge_pairs(gpu, half, np.random.default_rng(8), 4), 106, "long n=16 C=4096 P=98304")


@pytest.mark.parametrize("C,P,n,L,fused", [
    (4096, 4096, 128, 3200, True),      # whole items only, about 30 CTAs stream decode pages from the start
    (2048, 8192, 96, 4000, False),      # leftover items cut in two, side by side
    (2048, 12288, 35, 20000, True),     # about 60 leftover items cut in three: 180 pieces for the 98 CTAs that take them
    (2048, 16384, 47, 20000, False),    # about 60 leftover items cut in three to five, for 97 CTAs
    (2048, 0, 128, 3200, True),         # the decode pages are the longer part: the 256 short items run on about 30 CTAs
], ids=["whole_items", "two_pieces", "pieces_in_rounds", "more_pieces_in_rounds", "entries_on_few_ctas"])
def test_whole_rounds_of_items_beside_many_decode_pages(gpu, oracle, C, P, n, L, fused):
    """A chunk of at least one whole round of work items (one per SM) beside decode requests whose pages are a tenth of
    the launch or more: some CTAs take no chunk-prefill entry and stream decode pages from the start, the others share
    the items, and the items left over after their whole rounds are cut along the KV axis into pieces that may
    outnumber those CTAs (they are pulled from the counter over several rounds and merged by the last to arrive).
    The comments give what the plan does on a device of 148 SMs."""
    rng = np.random.default_rng(50 + C + P)
    lens = [L - (i * 37) % (L // 4) for i in range(n)]
    need = sum(-(-x // 16) for x in lens) + (P + C) // 16 + 64
    batch = W.make_batch(W.LLAMA, need, lens, P, C, rng)
    rows = gpu.boundary_rows(C, batch.shape.group) + list(range(0, 512, 7))   # the leftover items are the chunk's first rows
    pairs = sample_pairs(batch, np.random.default_rng(9), sorted(set(rows)), 12)
    run_case(gpu, oracle, batch, pairs, 150 + n, f"C={C} P={P} beside {n} decodes of up to {L} tokens", fused=fused)


@pytest.mark.parametrize("case", ["pieces_in_rounds", "chat", "one_long_request"])
def test_launches_stay_inside_the_workspace(gpu, oracle, case):
    """The context is created on the middle of a larger buffer whose first and last MiB hold a pattern: after an iteration
    that uses the scratch areas to the full (186 partial results of chunk-prefill pieces; the chat iteration; one request
    cut into about 150 units per KV head) the pattern is untouched and the results match the oracle."""
    import ctypes as C

    import torch

    from paper_2609_07883_b200 import binding as B

    class GuardedContext(B.Context):
        GUARD = 1 << 20

        def __init__(self, shape, num_pages, max_chunk, max_decode, max_pages):
            self.shape = shape
            self.layout = B.make_layout(shape, num_pages)
            self.device = torch.device("cuda", 0)
            self.nbytes = B.sw_workspace_bytes(self.layout, max_chunk, max_decode, max_pages)
            assert self.nbytes > 0
            self.whole = torch.full((self.nbytes + 2 * self.GUARD,), 0xA5, dtype=torch.uint8, device=self.device)
            self.workspace = self.whole[self.GUARD:self.GUARD + self.nbytes]
            handle = C.c_void_p()
            st = B._lib.sw_create(C.byref(self.layout), 0, self.workspace.data_ptr(), self.nbytes, max_chunk, max_decode,
                                  max_pages, C.byref(handle))
            assert st == B.SW_OK, B.sw_last_error()
            self.handle = handle

        def guards_intact(self):
            g, n = self.GUARD, self.nbytes
            return bool((self.whole[:g] == 0xA5).all().item()) and bool((self.whole[g + n:] == 0xA5).all().item())

    rng = np.random.default_rng(21)
    if case == "pieces_in_rounds":
        C_, P, n, L = 2048, 12288, 35, 20000
        lens = [L - (i * 37) % (L // 4) for i in range(n)]
        batch = W.make_batch(W.LLAMA, sum(-(-x // 16) for x in lens) + (P + C_) // 16 + 64, lens, P, C_, rng)
    elif case == "chat":
        batch = W.chat_batch(n=64, chunk_len=512, prefix_len=512, rng=rng)
    else:
        batch = W.make_batch(W.LLAMA, 20000 // 16 + 72, [20000], 0, 0, rng)
    total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
    ctx = GuardedContext(batch.shape, batch.num_pages, max(batch.chunk_len, 1), max(batch.num_decode, 1), total_pages + 16)
    pairs = sample_pairs(batch, np.random.default_rng(22), gpu.boundary_rows(batch.chunk_len, batch.shape.group)[::4], 8)
    for fused in (False, True):
        run_case(gpu, oracle, batch, pairs, 170, f"guarded workspace, {case}, fused={fused}", fused=fused, ctx=ctx)
        assert ctx.guards_intact(), f"{case}: a launch wrote outside the workspace"


def test_page_ids_above_two_to_the_twenty(gpu, oracle):
    """A 70 GB pool (1.1 M pages of 64 KB) with the live pages scattered over all of it: byte offsets pass 2^36."""
    import torch

    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    num_pages = (1 << 20) + 4096
    if free < num_pages * W.LLAMA.page_elems * 2 + (8 << 30):
        pytest.skip("not enough free device memory for the large pool")
    rng = np.random.default_rng(9)
    batch = W.make_batch(W.LLAMA, num_pages, [3000, 17, 700], 1000, 200, rng)
    assert int(max(batch.decode_pages.max(), batch.prefill_pages.max())) > (1 << 19)
    from paper_2609_07883_b200 import binding as B

    dev = torch.device("cuda", 0)
    sh = batch.shape
    ctx = B.Context(sh, num_pages, 200, 3, 512)
    db = B.DeviceBatch(batch, dev)
    pool = torch.zeros(num_pages * sh.page_elems, dtype=torch.bfloat16, device=dev)
    # fill only the live pages with data; the oracle works on a compact copy with renumbered pages
    live = np.concatenate([batch.decode_pages, batch.prefill_pages]).astype(np.int64)
    gen = torch.Generator(device=dev)
    gen.manual_seed(77)
    data = torch.randn(len(live), sh.page_elems, device=dev, generator=gen).to(torch.bfloat16)
    pool.view(num_pages, sh.page_elems)[torch.from_numpy(live).to(dev)] = data
    R = batch.num_rows
    q = torch.randn(R, sh.num_q_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    k_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    v_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    out = torch.zeros_like(q)
    B.sw_kv_append(ctx, pool, db, k_new, v_new)
    B.sw_mixed_attn_run(ctx, pool, db, q, out)
    torch.cuda.synchronize()
    assert B.sw_check_status(ctx, raise_on_error=False) == (0, 0)
    compact = W.MixedBatch(sh, len(live), batch.prefix_len, batch.chunk_len,
                           np.arange(len(batch.decode_pages), len(live), dtype=np.int32), batch.decode_kv_len,
                           batch.decode_page_indptr, np.arange(len(batch.decode_pages), dtype=np.int32))
    host_pool = gpu.torch_to_bits(data).reshape(-1).copy()
    assert oracle.kv_append(host_pool, compact, gpu.torch_to_bits(k_new), gpu.torch_to_bits(v_new)) == 0
    got_pages = gpu.torch_to_bits(pool.view(num_pages, sh.page_elems)[torch.from_numpy(live).to(dev)])
    assert np.array_equal(got_pages.reshape(-1), host_pool)            # append landed in the right far-away pages
    others = np.setdiff1d(rng.integers(0, num_pages, size=4096), live)                 # and nowhere else (sampled)
    untouched = pool.view(num_pages, sh.page_elems)[torch.from_numpy(others).to(dev)].view(torch.int16)
    assert int(torch.count_nonzero(untouched).item()) == 0
    ref, _, _ = oracle.mixed_attention(host_pool, compact, gpu.torch_to_bits(q))
    gpu.compare(W.bf16_bits_to_f64(gpu.torch_to_bits(out)).reshape(-1, sh.head_dim), None, ref, None, "far pages")

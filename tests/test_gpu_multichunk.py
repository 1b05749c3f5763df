"""Several prefill chunks (of different prompts) in one iteration, against the oracle run chunk by chunk: every chunk
is an attention problem of its own over its own prompt's pages, so the oracle's single-chunk routine, called once per
chunk and once for the decodes, defines the expected rows."""
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


def oracle_rows(oracle, batch, t):
    """Pool after the append and the expected out / lse rows, composed from single-chunk oracle calls."""
    sh = batch.shape
    pool = t["pool"].copy()
    out = np.zeros((batch.num_rows, sh.num_q_heads, sh.head_dim))
    lse = np.zeros((batch.num_rows, sh.num_q_heads))
    empty = np.zeros(0, np.int32)
    parts = []
    for P, C, row0, pages in batch.chunks():
        parts.append((W.MixedBatch(sh, batch.num_pages, P, C, pages, empty, np.zeros(1, np.int32), empty), row0, C))
    if batch.num_decode:
        parts.append((W.MixedBatch(sh, batch.num_pages, 0, 0, empty, batch.decode_kv_len, batch.decode_page_indptr,
                                   batch.decode_pages), batch.chunk_len, batch.num_decode))
    for b, row0, rows in parts:      # all appends first: a chunk may not read another's rows, but order is harmless
        assert oracle.kv_append(pool, b, t["k_new"][row0:row0 + rows], t["v_new"][row0:row0 + rows]) == 0
    for b, row0, rows in parts:
        o, l, _ = oracle.mixed_attention(pool, b, t["q"][row0:row0 + rows])
        out[row0:row0 + rows] = o.reshape(rows, sh.num_q_heads, sh.head_dim)
        lse[row0:row0 + rows] = l.reshape(rows, sh.num_q_heads)
    return pool, out, lse


CASES = {
    "two_small": (W.AttnShape(8, 2, 128), 300, [17, 300, 64], [(37, 91), (0, 50)]),
    "three_ragged_d64": (W.AttnShape(4, 4, 64), 400, [1, 16, 700], [(128, 300), (5, 1), (1000, 130)]),
    "prefill_only_eight": (W.TINY, 600, [], [(0, 40), (16, 16), (100, 257), (3, 5), (640, 64), (0, 1), (31, 33), (200, 100)]),
    "group8": (W.AttnShape(8, 1, 128), 300, [40, 500], [(64, 200), (300, 17)]),
    "llama_mixed": (W.LLAMA, 1200, [900, 2000, 333, 1500, 16], [(2048, 700), (0, 300), (512, 512)]),
    # chunks whose items are cut into different numbers of KV pieces: the end of a long prompt beside a new prompt,
    # three different counts, and counts trimmed because the pieces would outnumber the CTAs
    "long_end_new_start": (W.AttnShape(8, 2, 128), 400, [17, 300], [(3400, 70), (0, 50)]),
    "three_piece_counts": (W.AttnShape(8, 2, 128), 900, [64], [(8000, 100), (3300, 64), (0, 30)]),
    "pieces_trimmed_to_grid": (W.AttnShape(16, 16, 64), 1000, [100], [(9000, 300), (4000, 500)]),
    # more work items (176) than SMs beside 780 MB of decode pages: some CTAs take no chunk-prefill entry and stream
    # decode pages from the start, the whole rounds and the leftover pieces are shared by the others
    "entry_ctas_beside_decode_pages": (W.AttnShape(16, 8, 128), 12400, [16000 - 111 * i for i in range(12)],
                                       [(1000, 900), (0, 800), (300, 800)]),
}


@pytest.mark.parametrize("case", sorted(CASES))
@pytest.mark.parametrize("fused", [False, True])
def test_multi_chunk_iteration_matches_the_oracle(gpu, oracle, case, fused):
    shape, pages, lens, chunks = CASES[case]
    rng = np.random.default_rng(101)
    batch = W.make_multi_batch(shape, pages, lens, chunks, rng, name=case)
    assert batch.chunk_len == sum(c for _, c in chunks)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    if fused:
        r.iterate()
    else:
        r.append()
        r.attend()
    out, lse = r.results()
    assert r.status() == (0, 0)
    pool, ref, ref_lse = oracle_rows(oracle, batch, t)
    assert np.array_equal(gpu.torch_to_bits(r.pool), pool), "pool differs after append"
    gpu.compare(out.reshape(-1, shape.head_dim), lse.reshape(-1), ref.reshape(-1, shape.head_dim), ref_lse.reshape(-1),
                f"{case} fused={fused}")


def test_one_chunk_given_as_a_list_equals_the_single_chunk_batch(gpu, oracle):
    rng = np.random.default_rng(5)
    shape = W.AttnShape(8, 2, 128)
    single = W.make_batch(shape, 200, [100, 40], 77, 150, rng)
    multi = W.MixedBatch(shape, single.num_pages, single.prefix_len, single.chunk_len, single.prefill_pages,
                         single.decode_kv_len, single.decode_page_indptr, single.decode_pages,
                         chunk_prefix_lens=np.array([77], np.int32), chunk_lens=np.array([150], np.int32),
                         chunk_page_indptr=np.array([0, len(single.prefill_pages)], np.int32))
    t = W.host_tensors(single, rng)
    outs = []
    for b in (single, multi):
        r = gpu.Runner(b, t)
        r.iterate()
        o, l = r.results()
        assert r.status() == (0, 0)
        outs.append((o, l))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


def test_chunk_list_errors_are_refused_on_the_host(gpu):
    from paper_2609_07883_b200 import binding as B

    rng = np.random.default_rng(6)
    shape = W.AttnShape(8, 2, 128)
    batch = W.make_multi_batch(shape, 200, [30], [(0, 40), (16, 16)], rng)
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    bad = r.dbatch.struct
    keep = np.array([0, 3, 99], dtype=np.int32)                 # does not end at num_prefill_pages
    bad.chunk_page_indptr = keep.ctypes.data
    with pytest.raises(B.SwError):
        r.iterate()
    nine = W.make_multi_batch(shape, 400, [], [(0, 8)] * 9, rng)
    with pytest.raises(B.SwError):
        gpu.Runner(nine, W.host_tensors(nine, rng)).iterate()


def test_large_chunks_with_tail_pieces_sampled_rows(gpu, oracle):
    """152 work items on 148 SMs: the last four (the short second chunk's) are cut into KV pieces and merged; sampled
    (row, head) pairs of every chunk and of the decodes are compared."""
    rng = np.random.default_rng(202)
    shape = W.LLAMA
    chunks = [(20000, 1152), (9000, 64)]
    lens = [5000, 300, 12000]
    batch = W.make_multi_batch(shape, 4000, lens, chunks, rng, name="tail_pieces")
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    r.iterate()
    out, lse = r.results()
    assert r.status() == (0, 0)
    sh = shape
    pool = t["pool"].copy()
    empty = np.zeros(0, np.int32)
    parts = [(W.MixedBatch(sh, batch.num_pages, P, C, pages, empty, np.zeros(1, np.int32), empty), row0, C)
             for P, C, row0, pages in batch.chunks()]
    parts.append((W.MixedBatch(sh, batch.num_pages, 0, 0, empty, batch.decode_kv_len, batch.decode_page_indptr,
                               batch.decode_pages), batch.chunk_len, batch.num_decode))
    for b, row0, rows in parts:
        assert oracle.kv_append(pool, b, t["k_new"][row0:row0 + rows], t["v_new"][row0:row0 + rows]) == 0
    assert np.array_equal(gpu.torch_to_bits(r.pool), pool)
    for b, row0, rows in parts:
        local = sorted(set([0, rows - 1] + [int(x) for x in rng.integers(0, rows, size=10)]))
        pairs = np.array([(x, int(rng.integers(sh.num_q_heads))) for x in local], dtype=np.int32)
        ref, ref_lse, _ = oracle.mixed_attention(pool, b, t["q"][row0:row0 + rows], pairs=pairs)
        g = out[row0 + pairs[:, 0], pairs[:, 1]]
        gl = lse[row0 + pairs[:, 0], pairs[:, 1]]
        gpu.compare(g, gl, ref, ref_lse, f"tail pieces, rows from {row0}")


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_random_mixes_of_long_and_short_chunks(gpu, oracle, seed):
    """Two to eight chunks whose prefixes range from nothing to thousands of tokens: the chunks' items get different
    numbers of KV pieces (or none), in every order of long and short chunks, beside a few decodes."""
    rng = np.random.default_rng(700 + seed)
    shape = [W.AttnShape(8, 2, 128), W.AttnShape(4, 4, 64), W.AttnShape(8, 1, 128), W.AttnShape(16, 4, 64)][seed - 1]
    k = int(rng.integers(2, 9))
    chunks = [(int(rng.choice([0, 0, 700, 3500, 9000])) + int(rng.integers(0, 40)), int(rng.integers(1, 200)))
              for _ in range(k)]
    lens = [int(x) for x in rng.integers(1, 3000, size=int(rng.integers(0, 5)))]
    pages = sum(-(-(P + C) // 16) for P, C in chunks) + sum(-(-x // 16) for x in lens) + 16
    batch = W.make_multi_batch(shape, pages, lens, chunks, rng, name=f"random mix {seed}")
    t = W.host_tensors(batch, rng)
    r = gpu.Runner(batch, t)
    r.iterate()
    out, lse = r.results()
    assert r.status() == (0, 0)
    pool, ref, ref_lse = oracle_rows(oracle, batch, t)
    assert np.array_equal(gpu.torch_to_bits(r.pool), pool), "pool differs after append"
    gpu.compare(out.reshape(-1, shape.head_dim), lse.reshape(-1), ref.reshape(-1, shape.head_dim), ref_lse.reshape(-1),
                f"random mix {seed}: {chunks}")

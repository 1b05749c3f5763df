"""GPU parity with scores spread far apart: one key whose scaled score lies more than 100 above the rest (the softmax
puts all weight on it), planted where each part of the kernels has to cope with it, and whole-tensor variants with q
scaled by 8 and by 1/8.  Every case is compared with the fp64 oracle element by element (output, log-sum-exp) and must
hold no inf / NaN.

What the cases reach:
* chunk prefill, key in a later KV tile than the row's first: the row maximum grows by far more than the lazy-rescale
  threshold between two tiles, so the accumulator in TMEM is rescaled (by a factor that underflows to zero) and the row
  sum restarts; key in the first tile: every later tile contributes weights that underflow to zero.
* chunk prefill cut along the KV axis (few long items): the pieces' partial maxima differ by more than 100, all but
  one piece merge with weight zero.
* decode units: the same inside one unit (online rescale in registers) and across the splits of a request, with the
  last-ticket merge (a few splits) and the shared merge of requests cut into 24 splits or more.
"""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W

pytestmark = pytest.mark.gpu

SHAPE = W.AttnShape(8, 2, 128)
Q0 = 8.0        # element 0 of every query row
STRONG = 160.0  # element 0 of a planted key: adds Q0 * STRONG / sqrt(128) = 113 to its scaled score


@pytest.fixture(scope="module")
def gpu():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_07883_b200 import build

    build.build()
    from tests import gpu_util

    return gpu_util


def planter(batch, prompt_keys=(), decode_keys=()):
    """patch() for run_device_case: element 0 of every q row becomes Q0; element 0 of the listed keys becomes `strength`.
    prompt_keys: (position, kv head, strength) in the prefill prompt; decode_keys: (request, position, kv head, strength).
    Positions inside the chunk, and a request's last position, are rows of k_new (the append puts them into the pool)."""
    S = batch.shape.page_size
    P, C = batch.prefix_len, batch.chunk_len

    def patch(pool5, q, k_new, v_new):
        q[:, :, 0] = Q0
        for pos, kvh, strength in prompt_keys:
            if pos >= P:
                k_new[pos - P, kvh, 0] = strength
            else:
                pool5[int(batch.prefill_pages[pos // S]), 0, kvh, pos % S, 0] = strength
        for i, pos, kvh, strength in decode_keys:
            L = int(batch.decode_kv_len[i])
            if pos == L - 1:
                k_new[C + i, kvh, 0] = strength
            else:
                pages = batch.decode_pages[batch.decode_page_indptr[i]:batch.decode_page_indptr[i + 1]]
                pool5[int(pages[pos // S]), 0, kvh, pos % S, 0] = strength

    return patch


@pytest.mark.parametrize("where", ["first_tile", "middle_tile", "last_tile_in_chunk", "ladder"])
def test_prefill_row_with_a_dominant_key(gpu, oracle, where):
    """P=700, C=300: rows attend 701..1000 keys = 6 to 8 KV tiles of 128.  "ladder": three keys of growing strength in
    three different tiles, so the accumulator is rescaled more than once."""
    P, C = 700, 300
    batch = W.make_batch(SHAPE, (P + C) // 16 + 8, [], P, C, np.random.default_rng(11))
    keys = {"first_tile": [(5, 0, STRONG), (100, 1, STRONG)],
            "middle_tile": [(450, 0, STRONG), (520, 1, STRONG)],
            "last_tile_in_chunk": [(905, 0, STRONG), (990, 1, STRONG)],      # rows below the key never see it
            "ladder": [(60, 0, 48.0), (400, 0, 96.0), (950, 0, STRONG), (10, 1, 48.0), (700, 1, 112.0)]}[where]
    gpu.run_device_case(oracle, batch, None, 210, f"dominant key, prefill {where}", patch=planter(batch, prompt_keys=keys))


@pytest.mark.parametrize("pos", [3, 6100, 11990, 12040])
def test_prefill_pieces_with_a_dominant_key(gpu, oracle, pos):
    """P=12000, C=64: two work items of 95 KV tiles, each cut along the KV axis into pieces that are merged.  The
    dominant key sits in the first piece, a middle piece, the last tile of the prefix, or inside the chunk."""
    P, C = 12000, 64
    batch = W.make_batch(SHAPE, (P + C) // 16 + 40, [300, 5], P, C, np.random.default_rng(12))
    keys = [(pos, 0, STRONG), (pos, 1, 144.0)]
    gpu.run_device_case(oracle, batch, None, 220 + pos % 7, f"dominant key, prefill pieces pos={pos}",
                        patch=planter(batch, prompt_keys=keys))


def test_decode_units_with_dominant_keys(gpu, oracle):
    """Requests of 1 to 5000 tokens beside a small chunk: units of one page up to a few hundred tokens, requests cut into
    1 to about 40 splits.  Dominant keys in the first page, mid-context, on a split edge region, and in the token
    appended by this very iteration."""
    lens = [3000, 17, 700, 5000, 1, 129, 2048]
    batch = W.make_batch(SHAPE, sum(-(-x // 16) for x in lens) + 40, lens, 100, 40, np.random.default_rng(13))
    keys = [(0, 2, 0, STRONG), (0, 1500, 1, STRONG), (1, 16, 0, STRONG), (1, 0, 1, STRONG), (2, 699, 0, STRONG),
            (2, 350, 1, 144.0), (3, 4999, 1, STRONG), (3, 2560, 0, STRONG), (5, 128, 0, STRONG), (6, 1024, 0, 96.0),
            (6, 1100, 0, STRONG), (6, 2047, 1, STRONG)]
    for fused in (False, True):
        gpu.run_device_case(oracle, batch, None, 230, f"dominant keys, decode units (fused={fused})", fused=fused,
                            patch=planter(batch, decode_keys=keys))


@pytest.mark.parametrize("others", [0, 30])
def test_long_request_cut_into_many_splits(gpu, oracle, others):
    """One request of 20000 tokens.  Alone it is cut into about 150 units of 128 tokens per KV head (the shared merge of
    requests with 24 splits or more); beside 30 requests of the same length the units are about 45 pages and it has 28.
    The dominant key of KV head 0 sits mid-context, that of KV head 1 in the first page."""
    lens = [20000] * (1 + others)
    batch = W.make_batch(SHAPE, sum(-(-x // 16) for x in lens) + 40, lens, 0, 0, np.random.default_rng(14))
    keys = [(0, 9000, 0, STRONG), (0, 7, 1, STRONG)]
    if others:
        keys += [(5, 19999, 0, STRONG), (17, 12345, 1, 144.0)]
    pairs = None if not others else [(i, h) for i in (0, 5, 17, 29) for h in range(SHAPE.num_q_heads)]
    gpu.run_device_case(oracle, batch, pairs, 240, f"dominant key, one of {1 + others} long requests",
                        patch=planter(batch, decode_keys=keys))


@pytest.mark.parametrize("q_scale", [8.0, 0.125])
def test_whole_tensor_score_scale(gpu, oracle, q_scale):
    """q scaled by 8 (scores spread over tens of units: a few keys per row carry the weight, row maxima jump between
    tiles) and by 1/8 (a nearly uniform softmax over thousands of keys), chunk prefill and decodes in one launch."""
    lens = [900, 33, 4000]
    P, C = 1500, 260
    batch = W.make_batch(SHAPE, sum(-(-x // 16) for x in lens) + (P + C) // 16 + 8, lens, P, C, np.random.default_rng(15))
    gpu.run_device_case(oracle, batch, None, 250, f"q scaled by {q_scale}", fused=True, q_scale=q_scale)

"""Pins for the attention / paging half of the CPU oracle (no GPU).

Each test checks the oracle against something other than itself: a numpy float64 dense softmax written
with matrix products, closed forms, invariants and special cases.
"""
import numpy as np
import pytest

from paper_2609_07883_b200 import workloads as W


# ------------------------------------------------------------------------------------------------
# helpers (independent of the oracle's code: explicit 5-D views and matrix products)
# ------------------------------------------------------------------------------------------------
def pool_view(pool_bits, batch):
    sh = batch.shape
    return pool_bits.reshape(batch.num_pages, 2, sh.num_kv_heads, sh.page_size, sh.head_dim)


def gather_kv(pool_bits, batch, pages, kv_len):
    """K, V as float64 [kv_len][Hkv][d] gathered through the page list with a 5-D view."""
    pv = pool_view(pool_bits, batch)
    S = batch.shape.page_size
    k = np.stack([pv[pages[t // S], 0, :, t % S, :] for t in range(kv_len)])
    v = np.stack([pv[pages[t // S], 1, :, t % S, :] for t in range(kv_len)])
    return W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(v)


def numpy_row(qrow, K, V, scale):
    """softmax(q K^T scale) V for one row with numpy matrix products."""
    s = (K @ qrow) * scale
    w = np.exp(s - s.max())
    p = w / w.sum()
    return p @ V, s.max() + np.log(w.sum())


def numpy_mixed(pool_bits, batch, q_bits):
    sh = batch.shape
    g = sh.group
    scale = 1.0 / np.sqrt(sh.head_dim)
    q = W.bf16_bits_to_f64(q_bits)
    out = np.zeros((batch.num_rows, sh.num_q_heads, sh.head_dim))
    lse = np.zeros((batch.num_rows, sh.num_q_heads))
    if batch.chunk_len:
        K, V = gather_kv(pool_bits, batch, batch.prefill_pages, batch.prefix_len + batch.chunk_len)
        for j in range(batch.chunk_len):
            L = batch.prefix_len + j + 1
            for h in range(sh.num_q_heads):
                out[j, h], lse[j, h] = numpy_row(q[j, h], K[:L, h // g], V[:L, h // g], scale)
    for i in range(batch.num_decode):
        L = int(batch.decode_kv_len[i])
        pages = batch.decode_pages[batch.decode_page_indptr[i]:batch.decode_page_indptr[i + 1]]
        K, V = gather_kv(pool_bits, batch, pages, L)
        r = batch.chunk_len + i
        for h in range(sh.num_q_heads):
            out[r, h], lse[r, h] = numpy_row(q[r, h], K[:, h // g], V[:, h // g], scale)
    return out, lse


def small_batch(rng, shape=W.TINY, lens=(1, 17, 40), P=21, C=27, num_pages=24):
    return W.make_batch(shape, num_pages, list(lens), P, C, rng)


# ------------------------------------------------------------------------------------------------
# softmax rows sum to one; numpy dense softmax agreement on the tiny workload (brute force)
# ------------------------------------------------------------------------------------------------
def test_tiny_workload_matches_numpy_dense_and_rows_sum_to_one(oracle):
    rng = W.rng_for(0)
    batch = W.tiny_batch(rng)
    t = W.host_tensors(batch, rng)
    out, lse, psum = oracle.mixed_attention(t["pool"], batch, t["q"])
    assert np.all(np.abs(psum - 1.0) <= 1e-12)
    ref, ref_lse = numpy_mixed(t["pool"], batch, t["q"])
    sh = batch.shape
    out = out.reshape(batch.num_rows, sh.num_q_heads, sh.head_dim)
    assert np.max(np.abs(out - ref)) <= 1e-12
    assert np.max(np.abs(lse.reshape(ref_lse.shape) - ref_lse)) <= 1e-12


def test_pairs_selection_equals_full(oracle):
    rng = np.random.default_rng(5)
    batch = small_batch(rng)
    t = W.host_tensors(batch, rng)
    full, full_lse, _ = oracle.mixed_attention(t["pool"], batch, t["q"])
    Hq = batch.shape.num_q_heads
    pairs = np.array([[0, 0], [26, 7], [27, 3], [29, 5], [13, 2]], dtype=np.int32)
    sub, sub_lse, _ = oracle.mixed_attention(t["pool"], batch, t["q"], pairs=pairs)
    for i, (r, h) in enumerate(pairs):
        assert np.array_equal(sub[i], full[r * Hq + h])
        assert sub_lse[i] == full_lse[r * Hq + h]


# ------------------------------------------------------------------------------------------------
# paging: paged == dense unpaged (bit-exact); page permutation leaves the result bit-identical
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [W.TINY, W.AttnShape(4, 4, 32), W.AttnShape(6, 1, 16)])
def test_paged_equals_dense_unpaged_bit_exact(oracle, shape):
    rng = np.random.default_rng(11)
    T = 53
    batch = W.make_batch(shape, 16, [], 0, T, rng)
    q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
    k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    v = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    pool = W.normal_bf16_bits(rng, batch.num_pages * shape.page_elems)
    assert oracle.kv_append(pool, batch, k, v) == 0
    paged, paged_lse, _ = oracle.mixed_attention(pool, batch, q)
    dense, dense_lse = oracle.dense_causal(q, k, v, shape.num_q_heads, shape.num_kv_heads, shape.head_dim)
    assert np.array_equal(paged.reshape(dense.shape), dense)
    assert np.array_equal(paged_lse.reshape(dense_lse.shape), dense_lse)
    # and the dense routine against numpy matrix products
    qf, kf, vf = (W.bf16_bits_to_f64(x) for x in (q, k, v))
    g = shape.group
    for tt in (0, 1, 15, 16, 52):
        for h in range(shape.num_q_heads):
            ref, _ = numpy_row(qf[tt, h], kf[:tt + 1, h // g], vf[:tt + 1, h // g], 1 / np.sqrt(shape.head_dim))
            assert np.max(np.abs(dense[tt, h] - ref)) <= 1e-12


def test_page_permutation_leaves_output_bit_identical(oracle):
    rng = np.random.default_rng(3)
    shape = W.TINY
    T = 70
    q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
    k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    v = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    outs = []
    for seed in (1, 2):
        batch = W.make_batch(shape, 32, [], 0, T, np.random.default_rng(seed))
        pool = np.zeros(batch.num_pages * shape.page_elems, dtype=np.uint16)
        assert oracle.kv_append(pool, batch, k, v) == 0
        outs.append(oracle.mixed_attention(pool, batch, q)[0])
        last_pages = batch.prefill_pages
    assert not np.array_equal(last_pages, W.make_batch(shape, 32, [], 0, T, np.random.default_rng(1)).prefill_pages)
    assert np.array_equal(outs[0], outs[1])


# ------------------------------------------------------------------------------------------------
# chunk invariance: any split of a prompt gives the outputs of one unchunked causal prefill
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("split", [[96], [32, 32, 32], [1, 95], [17, 40, 39], [16] * 6, [50, 46]])
def test_chunk_invariance_bit_exact(oracle, split):
    rng = np.random.default_rng(21)
    shape = W.TINY
    T = sum(split)
    q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
    k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    v = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    dense, _ = oracle.dense_causal(q, k, v, shape.num_q_heads, shape.num_kv_heads, shape.head_dim)
    pages = np.random.default_rng(4).permutation(16)[: -(-T // 16)].astype(np.int32)
    pool = W.normal_bf16_bits(rng, 16 * shape.page_elems)  # garbage in unwritten slots must not matter
    P = 0
    got = []
    for c in split:
        batch = W.MixedBatch(shape, 16, P, c, pages[: -(-(P + c) // 16)].copy(), np.zeros(0, np.int32),
                             np.zeros(1, np.int32), np.zeros(0, np.int32))
        assert oracle.kv_append(pool, batch, k[P:P + c], v[P:P + c]) == 0
        o, _, _ = oracle.mixed_attention(pool, batch, q[P:P + c])
        got.append(o.reshape(c, shape.num_q_heads, shape.head_dim))
        P += c
    assert np.array_equal(np.concatenate(got), dense)


# ------------------------------------------------------------------------------------------------
# closed forms and special cases
# ------------------------------------------------------------------------------------------------
def _one_seq_batch(shape, T, num_pages=16, seed=9):
    return W.make_batch(shape, num_pages, [], 0, T, np.random.default_rng(seed))


def test_length_one_returns_v0_exactly(oracle):
    rng = np.random.default_rng(8)
    batch = small_batch(rng, lens=(1, 33), P=0, C=5)
    t = W.host_tensors(batch, rng)
    pool = t["pool"].copy()
    assert oracle.kv_append(pool, batch, t["k_new"], t["v_new"]) == 0
    out, _, _ = oracle.mixed_attention(pool, batch, t["q"])
    sh = batch.shape
    out = out.reshape(batch.num_rows, sh.num_q_heads, sh.head_dim)
    vnew = W.bf16_bits_to_f64(t["v_new"])
    g = sh.group
    for h in range(sh.num_q_heads):
        assert np.array_equal(out[0, h], vnew[0, h // g])  # prefill row at P=0, j=0
        assert np.array_equal(out[5, h], vnew[5, h // g])  # decode with L=1 sees only its own token


def test_v_all_ones_gives_ones_and_constant_k_gives_mean_of_v(oracle):
    rng = np.random.default_rng(2)
    shape = W.TINY
    T = 45
    batch = _one_seq_batch(shape, T)
    q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
    k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    ones = W.f32_to_bf16_bits(np.ones((T, shape.num_kv_heads, shape.head_dim), np.float32))
    pool = np.zeros(batch.num_pages * shape.page_elems, np.uint16)
    oracle.kv_append(pool, batch, k, ones)
    out, _, _ = oracle.mixed_attention(pool, batch, q)
    assert np.max(np.abs(out - 1.0)) <= 1e-12
    # K constant across tokens -> uniform weights -> running mean of V
    kc = np.broadcast_to(W.normal_bf16_bits(rng, 1, shape.num_kv_heads, shape.head_dim),
                         (T, shape.num_kv_heads, shape.head_dim)).copy()
    v = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    oracle.kv_append(pool, batch, kc, v)
    out, _, _ = oracle.mixed_attention(pool, batch, q)
    out = out.reshape(T, shape.num_q_heads, shape.head_dim)
    vf = W.bf16_bits_to_f64(v)
    for tt in (0, 7, 44):
        for h in range(shape.num_q_heads):
            assert np.max(np.abs(out[tt, h] - vf[:tt + 1, h // shape.group].mean(axis=0))) <= 1e-12


def test_causal_diagonal_is_inclusive_closed_form(oracle):
    """K == 0 and V[t][0] = t/256: the row at position p must give mean(0..p)/256 = p/512."""
    rng = np.random.default_rng(6)
    shape = W.TINY
    T = 200
    batch = _one_seq_batch(shape, T)
    q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
    k = np.zeros((T, shape.num_kv_heads, shape.head_dim), np.uint16)
    vf = np.zeros((T, shape.num_kv_heads, shape.head_dim), np.float32)
    vf[:, :, 0] = (np.arange(T, dtype=np.float32) / 256.0)[:, None]
    v = W.f32_to_bf16_bits(vf)
    assert np.array_equal(W.bf16_bits_to_f32(v), vf)  # exactly representable for t <= 256
    pool = np.zeros(batch.num_pages * shape.page_elems, np.uint16)
    oracle.kv_append(pool, batch, k, v)
    out, _, _ = oracle.mixed_attention(pool, batch, q)
    out = out.reshape(T, shape.num_q_heads, shape.head_dim)
    p = np.arange(T, dtype=np.float64)
    for h in range(shape.num_q_heads):
        assert np.max(np.abs(out[:, h, 0] - p / 512.0)) <= 1e-12
        assert np.max(np.abs(out[:, h, 1:])) == 0.0


def test_gqa_head_mapping(oracle):
    rng = np.random.default_rng(10)
    for shape in (W.TINY, W.AttnShape(12, 3, 16), W.AttnShape(4, 4, 16), W.AttnShape(8, 1, 16)):
        T = 20
        batch = _one_seq_batch(shape, T)
        q = W.normal_bf16_bits(rng, T, shape.num_q_heads, shape.head_dim)
        k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
        vf = np.zeros((T, shape.num_kv_heads, shape.head_dim), np.float32)
        vf += np.arange(shape.num_kv_heads, dtype=np.float32)[None, :, None]
        pool = np.zeros(batch.num_pages * shape.page_elems, np.uint16)
        oracle.kv_append(pool, batch, k, W.f32_to_bf16_bits(vf))
        out, _, _ = oracle.mixed_attention(pool, batch, q)
        out = out.reshape(T, shape.num_q_heads, shape.head_dim)
        for h in range(shape.num_q_heads):
            assert np.max(np.abs(out[:, h] - (h // shape.group))) <= 1e-12


def test_dominant_key_is_stable(oracle):
    """One key whose score exceeds the rest by > 100 takes the whole weight; no inf / nan."""
    rng = np.random.default_rng(12)
    shape = W.TINY
    T = 64
    batch = _one_seq_batch(shape, T)
    k = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    v = W.normal_bf16_bits(rng, T, shape.num_kv_heads, shape.head_dim)
    kf = W.bf16_bits_to_f32(k)
    star = 37
    qf = np.zeros((T, shape.num_q_heads, shape.head_dim), np.float32)
    for h in range(shape.num_q_heads):
        qf[:, h] = 64.0 * kf[star, h // shape.group]
    q = W.f32_to_bf16_bits(qf)
    pool = np.zeros(batch.num_pages * shape.page_elems, np.uint16)
    oracle.kv_append(pool, batch, k, v)
    out, lse, psum = oracle.mixed_attention(pool, batch, q)
    assert np.all(np.isfinite(out)) and np.all(np.isfinite(lse))
    out = out.reshape(T, shape.num_q_heads, shape.head_dim)
    vf = W.bf16_bits_to_f64(v)
    for h in range(shape.num_q_heads):
        assert np.max(np.abs(out[T - 1, h] - vf[star, h // shape.group])) <= 1e-9


# ------------------------------------------------------------------------------------------------
# KV append indexing
# ------------------------------------------------------------------------------------------------
def test_kv_append_matches_5d_view_scatter(oracle):
    rng = np.random.default_rng(14)
    batch = small_batch(rng, lens=(1, 16, 17, 48), P=21, C=27, num_pages=24)  # P mid-page, chunk crosses pages
    t = W.host_tensors(batch, rng)
    pool = t["pool"].copy()
    expect = t["pool"].copy()
    ev = pool_view(expect, batch)
    S = batch.shape.page_size
    for j in range(batch.chunk_len):
        pos = batch.prefix_len + j
        ev[batch.prefill_pages[pos // S], 0, :, pos % S, :] = t["k_new"][j]
        ev[batch.prefill_pages[pos // S], 1, :, pos % S, :] = t["v_new"][j]
    for i in range(batch.num_decode):
        pos = int(batch.decode_kv_len[i]) - 1
        pages = batch.decode_pages[batch.decode_page_indptr[i]:]
        r = batch.chunk_len + i
        ev[pages[pos // S], 0, :, pos % S, :] = t["k_new"][r]
        ev[pages[pos // S], 1, :, pos % S, :] = t["v_new"][r]
    assert oracle.kv_append(pool, batch, t["k_new"], t["v_new"]) == 0
    assert np.array_equal(pool, expect)
    assert not np.array_equal(pool, t["pool"])


def test_pool_index_is_64_bit_and_matches_strides(oracle):
    Hkv, S, d = 8, 16, 128
    strides = np.array([2 * Hkv * S * d, Hkv * S * d, S * d, d, 1], dtype=object)
    for page in (0, 1, (1 << 20) + 3, 1_831_053):
        for (x, h, r, e) in ((0, 0, 0, 0), (1, 7, 15, 127), (1, 0, 3, 64), (0, 5, 9, 1)):
            want = int(np.dot(np.array([page, x, h, r, e], dtype=object), strides))
            assert oracle.pool_index(page, x, h, r, e, Hkv, S, d) == want
    assert oracle.pool_index(1_831_053, 1, 7, 15, 127, Hkv, S, d) * 2 > (1 << 36)


def test_kv_append_rejects_bad_pages(oracle):
    rng = np.random.default_rng(15)
    batch = small_batch(rng)
    t = W.host_tensors(batch, rng)
    bad = W.MixedBatch(**{**batch.__dict__})
    bad.prefill_pages = batch.prefill_pages.copy()
    bad.prefill_pages[-1] = batch.num_pages  # one past the pool
    assert oracle.kv_append(t["pool"].copy(), bad, t["k_new"], t["v_new"]) == 2
    short = W.MixedBatch(**{**batch.__dict__})
    short.prefill_pages = batch.prefill_pages[:-1].copy()  # list too short for P+C
    assert oracle.kv_append(t["pool"].copy(), short, t["k_new"], t["v_new"]) == 2

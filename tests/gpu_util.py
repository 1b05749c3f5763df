"""Helpers shared by the GPU parity tests: run one mixed iteration through the C-ABI and compare with the oracle."""
from __future__ import annotations

import numpy as np

from paper_2609_07883_b200 import workloads as W

MAX_ABS = 2e-2      # bf16 inputs, fp32 accumulation: max |err|
MAX_REL_RMS = 1e-2  # ||gpu - ref||_2 / ||ref||_2
LSE_ABS = 1e-3


def bits_to_torch(bits: np.ndarray, device):
    import torch

    return torch.from_numpy(bits.view(np.int16).copy()).to(device).view(torch.bfloat16)


def torch_to_bits(t) -> np.ndarray:
    import torch

    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Runner:
    """Device buffers for one batch; runs append + attention through the binding."""

    def __init__(self, batch: W.MixedBatch, tensors: dict, device=0):
        import torch
        from paper_2609_07883_b200 import binding as B

        self.B = B
        self.batch = batch
        self.dev = torch.device("cuda", device)
        sh = batch.shape
        total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
        self.ctx = B.Context(sh, batch.num_pages, max(batch.chunk_len, 1), max(batch.num_decode, 1),
                             total_pages + 16, device=device)
        self.dbatch = B.DeviceBatch(batch, self.dev)
        self.pool = bits_to_torch(tensors["pool"], self.dev)
        self.q = bits_to_torch(tensors["q"], self.dev)
        self.k_new = bits_to_torch(tensors["k_new"], self.dev)
        self.v_new = bits_to_torch(tensors["v_new"], self.dev)
        self.out = torch.zeros_like(self.q)
        self.lse = torch.zeros(batch.num_rows, sh.num_q_heads, dtype=torch.float32, device=self.dev)

    def append(self):
        self.B.sw_kv_append(self.ctx, self.pool, self.dbatch, self.k_new, self.v_new)

    def attend(self):
        self.B.sw_mixed_attn_run(self.ctx, self.pool, self.dbatch, self.q, self.out, self.lse)

    def iterate(self):
        """Append and attention in one launch."""
        self.B.sw_mixed_iteration_run(self.ctx, self.pool, self.dbatch, self.k_new, self.v_new, self.q, self.out, self.lse)

    def status(self):
        return self.B.sw_check_status(self.ctx, raise_on_error=False)

    def results(self):
        import torch

        torch.cuda.synchronize()
        out = W.bf16_bits_to_f64(torch_to_bits(self.out))
        return out, self.lse.cpu().numpy().astype(np.float64)


def compare(gpu_out, gpu_lse, ref_out, ref_lse, what=""):
    """ref_* from the oracle (fp64).  Shapes: out [m][d], lse [m]."""
    assert np.all(np.isfinite(gpu_out)), f"{what}: non-finite output"
    err = np.abs(gpu_out - ref_out)
    rel = np.linalg.norm(gpu_out - ref_out) / max(np.linalg.norm(ref_out), 1e-30)
    assert err.max() <= MAX_ABS, f"{what}: max |err| {err.max():.4g} at {np.unravel_index(err.argmax(), err.shape)}"
    assert rel <= MAX_REL_RMS, f"{what}: relative RMS {rel:.4g}"
    if gpu_lse is not None:
        lerr = np.abs(gpu_lse - ref_lse)
        assert lerr.max() <= LSE_ABS, f"{what}: lse max |err| {lerr.max():.4g}"
    return float(err.max()), float(rel)


def run_device_case(oracle, batch, pairs, seed, what, fused=False, patch=None, q_scale=1.0, ctx=None, pool=None):
    """One iteration on inputs drawn on the device (pools too large to draw on the host), compared with the oracle on the
    (row, head) `pairs` (None = every pair).  The pool after the append is compared whole, bit for bit.

    fused: append and attention as one launch (else two).  patch(pool5, q, k_new, v_new): edits the device tensors in
    place before the run (pool5 is the [page][K|V][kv head][slot][element] view).  Returns (max |err|, relative RMS).
    """
    import torch

    from paper_2609_07883_b200 import binding as B

    dev = torch.device("cuda", 0)
    sh = batch.shape
    total_pages = int(batch.prefill_pages.shape[0] + batch.decode_pages.shape[0])
    if ctx is None:
        ctx = B.Context(sh, batch.num_pages, max(batch.chunk_len, 1), max(batch.num_decode, 1), total_pages + 16)
    db = B.DeviceBatch(batch, dev)
    if pool is None:
        pool = torch.empty(batch.num_pages * sh.page_elems, dtype=torch.bfloat16, device=dev)
        W.fill_normal_bf16_(pool, seed)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed + 1)
    R = batch.num_rows
    q = (torch.randn(R, sh.num_q_heads, sh.head_dim, device=dev, generator=gen) * q_scale).to(torch.bfloat16)
    k_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    v_new = torch.randn(R, sh.num_kv_heads, sh.head_dim, device=dev, generator=gen).to(torch.bfloat16)
    if patch is not None:
        patch(pool.view(batch.num_pages, 2, sh.num_kv_heads, sh.page_size, sh.head_dim), q, k_new, v_new)
    out = torch.zeros_like(q)
    lse = torch.zeros(R, sh.num_q_heads, dtype=torch.float32, device=dev)
    host_pool = torch_to_bits(pool)          # the inputs, before the append
    if fused:
        B.sw_mixed_iteration_run(ctx, pool, db, k_new, v_new, q, out, lse)
    else:
        B.sw_kv_append(ctx, pool, db, k_new, v_new)
        B.sw_mixed_attn_run(ctx, pool, db, q, out, lse)
    torch.cuda.synchronize()
    assert B.sw_check_status(ctx, raise_on_error=False) == (0, 0), f"{what}: device status"
    assert oracle.kv_append(host_pool, batch, torch_to_bits(k_new), torch_to_bits(v_new)) == 0
    assert np.array_equal(torch_to_bits(pool), host_pool), f"{what}: pool differs after append"
    got_all = W.bf16_bits_to_f64(torch_to_bits(out))
    lse_all = lse.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got_all)) and np.all(np.isfinite(lse_all)), f"{what}: non-finite output"
    if pairs is None:
        ref, ref_lse, _ = oracle.mixed_attention(host_pool, batch, torch_to_bits(q))
        return compare(got_all.reshape(-1, sh.head_dim), lse_all.reshape(-1), ref, ref_lse, what)
    pairs = np.asarray(pairs, dtype=np.int32)
    ref, ref_lse, _ = oracle.mixed_attention(host_pool, batch, torch_to_bits(q), pairs=pairs)
    return compare(got_all[pairs[:, 0], pairs[:, 1]], lse_all[pairs[:, 0], pairs[:, 1]], ref, ref_lse, what)


def boundary_rows(C, group, page=16):
    """Chunk rows (tokens) next to every edge that matters to the tiling: the first and last row, the rows on both sides
    of every 128-row tile edge (a tile holds 128 / group tokens, an item two tiles) and of every 128-key KV tile edge,
    and the rows around a sample of 16-token page edges."""
    rows = {0, 1, C - 2, C - 1}
    tile_tokens = max(1, 128 // group)
    for edge in range(tile_tokens, C, tile_tokens):
        rows.update((edge - 1, edge))
    for edge in range(128, C, 128):
        rows.update((edge - 1, edge, edge + 1))
    for edge in list(range(page, min(C, 8 * page), page)) + [C // 2 // page * page + page, (C - 1) // page * page]:
        rows.update((edge - 1, edge))
    return sorted(r for r in rows if 0 <= r < C)

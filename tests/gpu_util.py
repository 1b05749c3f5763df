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

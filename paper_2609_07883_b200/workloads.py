"""Seeded synthetic inputs for the mixed prefill-chunk + decode attention iteration.

This module serves both the CPU oracle's tests and the CUDA path's tests / bench.  It draws shapes,
lengths, page permutations and tensor values; it contains none of the method's arithmetic (no
attention, no paging index formula, no chunk choice).  bf16 values travel as uint16 bit patterns so
that numpy can hold them and both sides see the same bits.

Workload recipes (the paper's workloads are synthetic length distributions; these restate them as
single-iteration snapshots):

* tiny     8 q heads / 2 KV heads / d=64, 64-page pool, decodes {64,100,180,256}, chunk C=128 at P=256
* chat     32/8/128, n decodes with contexts uniform in [256, 2048], chunk C at P=512 of a 1024 prompt
* mixed    32/8/128, 128 decodes with contexts lognormal(median 2048, sigma 1) clipped to [128, 16384]
* long     32/8/128, 16 decodes with contexts uniform in [32768, 131072], chunk at P=98304
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED_BASE = 0x78830000


# --------------------------------------------------------------------------------------------
# bf16 <-> float bit handling (representation only)
# --------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even) and return the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounding = ((u >> 16) & 1) + 0x7FFF
    out = ((u + rounding) >> 16).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------------------------
# shapes and batches
# --------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class AttnShape:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def page_elems(self) -> int:
        """bf16 elements of one page (K and V, all KV heads)."""
        return 2 * self.num_kv_heads * self.page_size * self.head_dim

    @property
    def token_bytes(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2


TINY = AttnShape(8, 2, 64)
LLAMA = AttnShape(32, 8, 128)


@dataclass
class MixedBatch:
    """One mixed iteration: a prefill chunk [P, P+C) of one prompt plus n decode requests.

    ``decode_kv_len[i]`` is the number of keys request i attends, i.e. its context *including* the
    token whose K/V row is appended in this iteration.  Page lists hold pool page ids.
    """

    shape: AttnShape
    num_pages: int
    prefix_len: int
    chunk_len: int
    prefill_pages: np.ndarray  # int32 [ceil((P+C)/page)]
    decode_kv_len: np.ndarray  # int32 [n]
    decode_page_indptr: np.ndarray  # int32 [n+1]
    decode_pages: np.ndarray  # int32 [indptr[n]]
    name: str = ""
    meta: dict = field(default_factory=dict)
    # Several prefill chunks (of different prompts) in one iteration: chunk j has chunk_lens[j] tokens at prefix
    # chunk_prefix_lens[j]; its rows follow chunk j-1's and its prompt's pages are
    # prefill_pages[chunk_page_indptr[j]:chunk_page_indptr[j+1]].  chunk_len is then the sum of the chunk lengths and
    # prefix_len the first chunk's.  None = the single chunk (prefix_len, chunk_len).
    chunk_prefix_lens: np.ndarray | None = None
    chunk_lens: np.ndarray | None = None
    chunk_page_indptr: np.ndarray | None = None

    def chunks(self):
        """[(P, C, first row, page list)] of the iteration's prefill chunks (one entry for a single-chunk batch)."""
        if self.chunk_lens is None:
            return [(self.prefix_len, self.chunk_len, 0, self.prefill_pages)] if self.chunk_len > 0 else []
        out, row = [], 0
        for j, (P, C) in enumerate(zip(self.chunk_prefix_lens, self.chunk_lens)):
            out.append((int(P), int(C), row, self.prefill_pages[self.chunk_page_indptr[j]:self.chunk_page_indptr[j + 1]]))
            row += int(C)
        return out

    @property
    def num_decode(self) -> int:
        return int(self.decode_kv_len.shape[0])

    @property
    def num_rows(self) -> int:
        return self.chunk_len + self.num_decode

    @property
    def total_decode_ctx(self) -> int:
        return int(self.decode_kv_len.astype(np.int64).sum())


def _cdiv(a: int, b: int) -> int:
    return -(-a // b)


def make_batch(shape: AttnShape, num_pages: int, decode_lens, prefix_len: int, chunk_len: int,
               rng: np.random.Generator, name: str = "") -> MixedBatch:
    """Deal distinct, randomly permuted pool pages to the decodes (in order) and then to the prompt."""
    decode_lens = np.asarray(decode_lens, dtype=np.int32).reshape(-1)
    S = shape.page_size
    per_req = [_cdiv(int(L), S) for L in decode_lens]
    n_pf = _cdiv(prefix_len + chunk_len, S) if (prefix_len + chunk_len) > 0 else 0
    need = sum(per_req) + n_pf
    if need > num_pages:
        raise ValueError(f"batch needs {need} pages, pool has {num_pages}")
    if num_pages <= (1 << 22):
        ids = rng.permutation(num_pages)[:need]
    else:
        ids = rng.choice(num_pages, size=need, replace=False)
    ids = ids.astype(np.int32)
    indptr = np.zeros(len(per_req) + 1, dtype=np.int32)
    indptr[1:] = np.cumsum(per_req)
    return MixedBatch(shape=shape, num_pages=int(num_pages), prefix_len=int(prefix_len),
                      chunk_len=int(chunk_len), prefill_pages=ids[indptr[-1]:].copy(),
                      decode_kv_len=decode_lens.copy(), decode_page_indptr=indptr,
                      decode_pages=ids[:indptr[-1]].copy(), name=name)


def make_multi_batch(shape: AttnShape, num_pages: int, decode_lens, chunks, rng: np.random.Generator,
                     name: str = "") -> MixedBatch:
    """As ``make_batch`` with several prefill chunks ``[(prefix_len, chunk_len), ...]``, each of its own prompt."""
    chunks = [(int(P), int(C)) for P, C in chunks]
    S = shape.page_size
    base = make_batch(shape, num_pages, decode_lens, 0, 0, rng, name=name)
    used = set(int(x) for x in base.decode_pages)
    free = np.array([i for i in rng.permutation(num_pages) if int(i) not in used], dtype=np.int32)
    per = [_cdiv(P + C, S) for P, C in chunks]
    if sum(per) > len(free):
        raise ValueError(f"batch needs {sum(per)} more pages, pool has {len(free)} free")
    indptr = np.zeros(len(chunks) + 1, dtype=np.int32)
    indptr[1:] = np.cumsum(per)
    return MixedBatch(shape=shape, num_pages=int(num_pages), prefix_len=chunks[0][0], chunk_len=sum(C for _, C in chunks),
                      prefill_pages=free[:indptr[-1]].copy(), decode_kv_len=base.decode_kv_len,
                      decode_page_indptr=base.decode_page_indptr, decode_pages=base.decode_pages, name=name,
                      chunk_prefix_lens=np.array([P for P, _ in chunks], dtype=np.int32),
                      chunk_lens=np.array([C for _, C in chunks], dtype=np.int32), chunk_page_indptr=indptr)


def normal_bf16_bits(rng: np.random.Generator, *size: int) -> np.ndarray:
    """N(0,1) drawn in float32 and rounded to bf16 bits."""
    return f32_to_bf16_bits(rng.standard_normal(size=size, dtype=np.float32))


def host_tensors(batch: MixedBatch, rng: np.random.Generator, with_pool: bool = True) -> dict:
    """Random q / k_new / v_new rows (and the whole pool for small pools), all as bf16 bits.

    Row order everywhere: rows 0..C-1 are the prefill chunk tokens, rows C..C+n-1 the decode tokens.
    """
    sh = batch.shape
    R = batch.num_rows
    out = {
        "q": normal_bf16_bits(rng, R, sh.num_q_heads, sh.head_dim),
        "k_new": normal_bf16_bits(rng, R, sh.num_kv_heads, sh.head_dim),
        "v_new": normal_bf16_bits(rng, R, sh.num_kv_heads, sh.head_dim),
    }
    if with_pool:
        out["pool"] = normal_bf16_bits(rng, batch.num_pages * sh.page_elems)
    return out


# --------------------------------------------------------------------------------------------
# the named workloads
# --------------------------------------------------------------------------------------------
def rng_for(config_index: int, salt: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(SEED_BASE + config_index + (salt << 8)))


def tiny_batch(rng: np.random.Generator | None = None) -> MixedBatch:
    rng = rng or rng_for(0)
    return make_batch(TINY, 64, [64, 100, 180, 256], 256, 128, rng, name="tiny")


def chat_batch(n: int = 64, chunk_len: int = 512, prefix_len: int = 512, slack_pages: int = 64,
               rng: np.random.Generator | None = None) -> MixedBatch:
    rng = rng or rng_for(1)
    lens = rng.integers(256, 2048, size=n, endpoint=True)
    need = int(sum(_cdiv(int(x), 16) for x in lens)) + _cdiv(prefix_len + chunk_len, 16)
    return make_batch(LLAMA, need + slack_pages, lens, prefix_len, chunk_len, rng, name=f"chat_n{n}_C{chunk_len}")


def mixed_lens(n: int, rng: np.random.Generator) -> np.ndarray:
    raw = np.floor(rng.lognormal(mean=np.log(2048.0), sigma=1.0, size=n))
    return np.clip(raw, 128, 16384).astype(np.int32)


def mixed_batch(chunk_len: int, prefix_len: int, n: int = 128, slack_pages: int = 256,
                rng: np.random.Generator | None = None) -> MixedBatch:
    rng = rng or rng_for(2)
    lens = mixed_lens(n, rng)
    need = int(sum(_cdiv(int(x), 16) for x in lens)) + _cdiv(prefix_len + chunk_len, 16)
    return make_batch(LLAMA, need + slack_pages, lens, prefix_len, chunk_len, rng,
                      name=f"mixed_C{chunk_len}_P{prefix_len}")


def long_batch(chunk_len: int, prefix_len: int = 98304, n: int = 16, num_pages: int | None = None,
               rng: np.random.Generator | None = None) -> MixedBatch:
    rng = rng or rng_for(3)
    lens = rng.integers(32768, 131072, size=n, endpoint=True)
    need = int(sum(_cdiv(int(x), 16) for x in lens)) + _cdiv(prefix_len + chunk_len, 16)
    if num_pages is None:
        num_pages = need + 1024
    return make_batch(LLAMA, int(num_pages), lens, prefix_len, chunk_len, rng,
                      name=f"long_C{chunk_len}_P{prefix_len}")


# --------------------------------------------------------------------------------------------
# request traces for the bursty controller loop
# --------------------------------------------------------------------------------------------
def bursty_trace(num_requests: int = 2000, rate_low: float = 2.0, rate_high: float = 20.0,
                 mean_dwell_s: float = 10.0, prompt_median: float = 1500.0, prompt_sigma: float = 1.0,
                 prompt_clip=(32, 32768), mean_output: float = 200.0,
                 rng: np.random.Generator | None = None) -> dict:
    """2-state Markov-modulated Poisson arrivals (starting in the low state), lognormal prompt
    lengths and geometric output lengths.  Times are int64 nanoseconds."""
    rng = rng or rng_for(4)
    arrivals = np.empty(num_requests, dtype=np.int64)
    t = 0.0
    state_high = False
    state_end = rng.exponential(mean_dwell_s)
    i = 0
    while i < num_requests:
        rate = rate_high if state_high else rate_low
        gap = rng.exponential(1.0 / rate)
        if t + gap >= state_end:
            # memoryless: jump to the switch point and redraw in the new state
            t = state_end
            state_high = not state_high
            state_end = t + rng.exponential(mean_dwell_s)
            continue
        t += gap
        arrivals[i] = int(round(t * 1e9))
        i += 1
    prompts = np.clip(np.floor(rng.lognormal(np.log(prompt_median), prompt_sigma, size=num_requests)),
                      prompt_clip[0], prompt_clip[1]).astype(np.int32)
    outputs = rng.geometric(1.0 / mean_output, size=num_requests).astype(np.int32)
    return {"arrival_ns": arrivals, "prompt_len": prompts, "output_len": outputs}


# --------------------------------------------------------------------------------------------
# request traces of the simulator study (Sec. 4.2): 1,000 requests, clipped log-normal lengths
# --------------------------------------------------------------------------------------------
# Offered rate (requests/s), TTFT SLO (ms) and length medians are the paper's; the log-normal sigmas, the clipping
# ranges and the burst parameters are not stated there and are chosen here (sigma 0.5 for prompts and outputs, which
# brings the static policies' P99 TTFT and TPOT on the mixed workload close to the published ones; prompts clipped to
# [16, 8192], outputs to [4, 1024]; bursty: 20 and 120 requests/s with 1 s mean dwell, which gives the stated
# 70 requests/s on average).
STUDY = {
    "chat": {"rate": 110.0, "ttft_slo_ms": 1000.0, "prompt_median": (256.0,), "prompt_mix": (1.0,), "output_median": 96.0},
    "mixed": {"rate": 90.0, "ttft_slo_ms": 1000.0, "prompt_median": (256.0, 1800.0), "prompt_mix": (0.7, 0.3),
              "output_median": 100.0},
    "long": {"rate": 60.0, "ttft_slo_ms": 5000.0, "prompt_median": (1800.0,), "prompt_mix": (1.0,), "output_median": 180.0},
    "bursty": {"rate": 70.0, "ttft_slo_ms": 1500.0, "prompt_median": (256.0, 1800.0), "prompt_mix": (0.7, 0.3),
               "output_median": 100.0, "rates": (20.0, 120.0), "mean_dwell_s": 1.0},
}


def study_trace(workload: str, seed: int, num_requests: int = 1000, prompt_sigma: float = 0.5, output_sigma: float = 0.5,
                prompt_clip=(16, 8192), output_clip=(4, 1024)) -> dict:
    """One trace of a study workload: exponential interarrival times (two-state for "bursty"), prompts drawn from the
    workload's mixture of clipped log-normals, outputs from one clipped log-normal.  Times are int64 nanoseconds."""
    cfg = STUDY[workload]
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + 9000 + 97 * seed + sorted(STUDY).index(workload)))
    if "rates" in cfg:
        arrivals = bursty_trace(num_requests, cfg["rates"][0], cfg["rates"][1], cfg["mean_dwell_s"], rng=rng)["arrival_ns"]
    else:
        arrivals = np.round(np.cumsum(rng.exponential(1.0 / cfg["rate"], size=num_requests)) * 1e9).astype(np.int64)
    which = rng.choice(len(cfg["prompt_mix"]), size=num_requests, p=np.asarray(cfg["prompt_mix"]))
    medians = np.asarray(cfg["prompt_median"])[which]
    prompts = np.clip(np.floor(medians * np.exp(prompt_sigma * rng.standard_normal(num_requests))), *prompt_clip)
    outputs = np.clip(np.floor(cfg["output_median"] * np.exp(output_sigma * rng.standard_normal(num_requests))), *output_clip)
    return {"arrival_ns": arrivals, "prompt_len": prompts.astype(np.int32), "output_len": outputs.astype(np.int32)}


# --------------------------------------------------------------------------------------------
# device-side fills for pools too large to draw on the host (torch imported lazily)
# --------------------------------------------------------------------------------------------
def fill_normal_bf16_(tensor, seed: int, slab_elems: int = 1 << 28) -> None:
    """Fill a (possibly huge) bf16 torch tensor in place with N(0,1), slab by slab, from one seed."""
    import torch

    gen = torch.Generator(device=tensor.device)
    gen.manual_seed(int(seed))
    flat = tensor.view(-1)
    for start in range(0, flat.numel(), slab_elems):
        flat[start:start + slab_elems].normal_(0.0, 1.0, generator=gen)

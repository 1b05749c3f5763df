"""ctypes front end of the CPU oracle (``sw_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the bench's CPU legs, never by the
CUDA library or its binding.  It compiles ``sw_oracle.c`` with gcc on first use and marshals numpy
arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "sw_oracle.c"
_LIB = _HERE / "libsw_oracle.so"
_lib = None

F_NO_PREFILL, F_NO_DECODE, F_DECODE_INFEASIBLE, F_CAPPED = 1, 2, 4, 8
INF = (1 << 63) - 1


# SW_ORACLE_SANITIZE=1 builds and loads the same source instrumented with -fsanitize=address,undefined (the sanitizer
# run of the CPU tests; the process must have been started with the sanitizer runtimes preloaded).
_SANITIZE = os.environ.get("SW_ORACLE_SANITIZE", "") not in ("", "0")
_LIB_ASAN = _HERE / "libsw_oracle_asan.so"


def build(force: bool = False, sanitize: bool = False) -> Path:
    target = _LIB_ASAN if sanitize else _LIB
    flags = (["-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer"]
             if sanitize else ["-O2"])
    if force or not target.exists() or target.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = target.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(["gcc"] + flags + ["-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, target)
    return target


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build(sanitize=_SANITIZE)))
        _lib.swo_pool_index.restype = C.c_int64
        _lib.swo_pool_index.argtypes = [C.c_int64] + [C.c_int] * 7
        _lib.swo_analytic_cost_ns.restype = C.c_int64
        _lib.swo_analytic_cost_ns.argtypes = [C.c_int64, C.c_int64]
        _lib.swo_num_threads.restype = C.c_int
    return _lib


def _p(a, ctype):
    if a is None:
        return None
    return a.ctypes.data_as(C.POINTER(ctype))


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def num_threads() -> int:
    return int(lib().swo_num_threads())


def pool_index(page, x, kvh, slot, e, Hkv, S, d) -> int:
    return int(lib().swo_pool_index(int(page), x, kvh, slot, e, Hkv, S, d))


def kv_append(pool, batch, k_new, v_new) -> int:
    """In-place scatter into ``pool`` (uint16 bits).  Returns the oracle's status code."""
    sh = batch.shape
    pool = _u16(pool)
    pf = _i32(batch.prefill_pages)
    return int(lib().swo_kv_append(
        _p(pool, C.c_uint16), C.c_int64(batch.num_pages), sh.num_kv_heads, sh.page_size, sh.head_dim,
        _p(_u16(k_new), C.c_uint16), _p(_u16(v_new), C.c_uint16),
        batch.prefix_len, batch.chunk_len, _p(pf, C.c_int32), int(pf.shape[0]),
        batch.num_decode, _p(_i32(batch.decode_kv_len), C.c_int32),
        _p(_i32(batch.decode_page_indptr), C.c_int32), _p(_i32(batch.decode_pages), C.c_int32)))


def mixed_attention(pool, batch, q, pairs=None, scale: float = 0.0, threads: int = 0):
    """Attention of a mixed iteration in fp64.

    pairs=None evaluates every (row, head); otherwise ``pairs`` is an int array [m][2] of (row, head).
    Returns (out [m][d] float64, lse [m] float64, psum [m] float64); with pairs=None the first axis is
    (C+n)*Hq in row-major order.
    """
    sh = batch.shape
    pool, q = _u16(pool), _u16(q)
    if pairs is None:
        m = batch.num_rows * sh.num_q_heads
        pp = None
    else:
        pp = _i32(pairs).reshape(-1, 2)
        m = pp.shape[0]
    out = np.zeros((m, sh.head_dim), dtype=np.float64)
    lse = np.zeros(m, dtype=np.float64)
    psum = np.zeros(m, dtype=np.float64)
    pf = _i32(batch.prefill_pages)
    dl, ip, dp = _i32(batch.decode_kv_len), _i32(batch.decode_page_indptr), _i32(batch.decode_pages)
    rc = lib().swo_mixed_attention(
        _p(pool, C.c_uint16), C.c_int64(batch.num_pages), sh.num_q_heads, sh.num_kv_heads, sh.page_size,
        sh.head_dim, C.c_double(scale), batch.prefix_len, batch.chunk_len, _p(pf, C.c_int32),
        int(pf.shape[0]), batch.num_decode, _p(dl, C.c_int32), _p(ip, C.c_int32), _p(dp, C.c_int32),
        _p(q, C.c_uint16), _p(pp, C.c_int32), C.c_int64(m), _p(out, C.c_double), _p(lse, C.c_double),
        _p(psum, C.c_double), int(threads))
    if rc != 0:
        raise RuntimeError(f"oracle swo_mixed_attention failed with status {rc}")
    return out, lse, psum


def dense_causal(q, k, v, Hq, Hkv, d, scale: float = 0.0):
    q, k, v = _u16(q), _u16(k), _u16(v)
    T = q.shape[0]
    out = np.zeros((T, Hq, d), dtype=np.float64)
    lse = np.zeros((T, Hq), dtype=np.float64)
    rc = lib().swo_dense_causal(_p(q, C.c_uint16), _p(k, C.c_uint16), _p(v, C.c_uint16), T, Hq, Hkv, d,
                                C.c_double(scale), _p(out, C.c_double), _p(lse, C.c_double))
    if rc != 0:
        raise RuntimeError(f"oracle swo_dense_causal failed with status {rc}")
    return out, lse


class Table:
    """Raw cost table held as numpy arrays (the oracle keeps no opaque object)."""

    def __init__(self, n_grid, ctx_grid, prefix_grid, chunk_grid, cost_ns, interp: bool = False):
        self.n_grid, self.ctx_grid = _i32(n_grid), _i64(ctx_grid)
        self.prefix_grid, self.chunk_grid = _i32(prefix_grid), _i32(chunk_grid)
        shape = (len(self.n_grid), len(self.ctx_grid), len(self.prefix_grid), len(self.chunk_grid))
        self.cost = _i64(cost_ns).reshape(shape).copy()
        self.interp = bool(interp)

    def cummax(self) -> "Table":
        s = self.cost.shape
        lib().swo_cummax(_p(self.cost, C.c_int64), s[0], s[1], s[2], s[3])
        return self

    def _grid_args(self):
        return (_p(self.n_grid, C.c_int32), len(self.n_grid), _p(self.ctx_grid, C.c_int64), len(self.ctx_grid),
                _p(self.prefix_grid, C.c_int32), len(self.prefix_grid), _p(self.chunk_grid, C.c_int32),
                len(self.chunk_grid), _p(self.cost, C.c_int64), int(self.interp))

    def lookup(self, n, ctx, prefix, c) -> int:
        out = C.c_int64(0)
        rc = lib().swo_cost_lookup(*self._grid_args(), C.c_int64(n), C.c_int64(ctx), C.c_int64(prefix),
                                   C.c_int64(c), C.byref(out))
        if rc != 0:
            raise IndexError(f"oracle cost lookup out of range (status {rc})")
        return int(out.value)

    def choose(self, now_ns, deadlines_ns, total_ctx, prefix_len, remaining, c_max=4096, quantum=1,
               margin_abs_ns=0, margin_ppm=0):
        """Brute-force Eq. (1).  Returns (chunk, flags, budget_ns)."""
        dl = _i64(deadlines_ns)
        chunk, flags, budget = C.c_int32(0), C.c_int32(0), C.c_int64(0)
        rc = lib().swo_choose_bruteforce(*self._grid_args(), C.c_int64(margin_abs_ns), C.c_int32(margin_ppm),
                                         C.c_int32(c_max), C.c_int32(quantum), C.c_int64(now_ns),
                                         _p(dl, C.c_int64), C.c_int32(len(dl)), C.c_int64(total_ctx),
                                         C.c_int32(prefix_len), C.c_int32(remaining), C.byref(chunk),
                                         C.byref(flags), C.byref(budget))
        if rc != 0:
            raise IndexError(f"oracle chooser failed (status {rc})")
        return int(chunk.value), int(flags.value), int(budget.value)


def choose_first_fit(table: Table, now_ns, deadlines_ns, total_ctx, prefix_lens, remaining, c_max=4096, quantum=1,
                     margin_abs_ns=0, margin_ppm=0, max_chunks=8):
    """Several prefills in one iteration by first fit (Sec. 3.3, "Prefill batching"), written out by exhaustive scan.

    Pending requests are taken oldest first.  With t tokens already admitted and the sum S of the admitted requests'
    prefix lengths, request j may add c tokens if T^(n, ctx, S + prefix_j, t + c) + delta <= B (the prediction for the
    total number of prefill tokens at the summed prefix bounds both the arithmetic and the K/V traffic of the separate
    chunks from above).  The largest such c in {multiples of the quantum, <= L_j} with L_j = min(C_max - t,
    remaining_j) is taken; a request that is admitted whole is followed by the next one, a request that is cut (or
    gets nothing) ends the list.  Without active decodes there is no deadline: requests are admitted whole up to
    C_max tokens.  Returns (chunks list, budget_ns)."""
    dl = [int(x) for x in deadlines_ns]
    n = len(dl)
    budget = max(0, min(dl) - int(now_ns)) if n else 0
    chunks, t, prefix_sum = [], 0, 0
    q = max(1, int(quantum))

    def cost(prefix, c):
        raw = table.lookup(n, total_ctx, prefix, c)
        if raw >= INF:
            return INF
        return raw + margin_abs_ns + -(-raw * margin_ppm // 1_000_000)

    for j in range(min(len(remaining), max_chunks)):
        L = min(c_max - t, int(remaining[j]))
        if L <= 0:
            break
        if n == 0:
            c = L - L % q
        else:
            c = 0
            for cand in range(L - L % q, 0, -q):
                if cost(prefix_sum + int(prefix_lens[j]), t + cand) <= budget:
                    c = cand
                    break
        if c == 0:
            break
        chunks.append(c)
        t += c
        prefix_sum += int(prefix_lens[j])
        if c < int(remaining[j]):
            break
    return chunks, budget


def analytic_cost_ns(n: int, c: int) -> int:
    return int(lib().swo_analytic_cost_ns(int(n), int(c)))


def analytic_table(n_values, c_max: int) -> Table:
    """The analytic model tabulated at every integer chunk 0..c_max for the given decode batch sizes."""
    n_values = sorted(int(x) for x in n_values)
    chunk_grid = np.arange(0, c_max + 1, dtype=np.int32)
    cost = np.zeros((len(n_values), 1, 1, len(chunk_grid)), dtype=np.int64)
    for a, n in enumerate(n_values):
        for e, c in enumerate(chunk_grid):
            cost[a, 0, 0, e] = analytic_cost_ns(n, int(c))
    return Table(n_values, [1 << 40], [1 << 30], chunk_grid, cost)


# --------------------------------------------------------------------------------------------
# telemetry residuals (Sec. 3.3 "Prediction error"; Sec. 5.1; Table 1 "Telemetry") — plain Python
# --------------------------------------------------------------------------------------------
class ResidualTable:
    """Empirical high-percentile residual table: the margin delta(n, c) of Sec. 3.3 and the fallback signal of
    Sec. 5.1, written out as their definitions.

    * residual of an iteration = max(0, observed - predicted) (one-sided: only under-prediction costs a deadline);
    * iterations are bucketed by (n, c): a value falls into the first bucket whose upper edge is >= it, values
      beyond the last edge into the last bucket; a bucket keeps its most recent ``window`` residuals;
    * percentile = nearest rank: the ceil(p * N)-th smallest of the N kept residuals (at least the first);
    * a bucket with fewer than ``min_samples`` residuals contributes ``floor_ns``;
    * delta(n, c) = the largest bucket percentile over all buckets (i, j) with i <= bucket(n) and j <= bucket(c), so
      that the margin is nondecreasing in n and in c (the feasibility test must stay monotone, Proposition 1);
    * the fallback signal is delta(n, c) > the configured margin.
    """

    def __init__(self, n_edges, c_edges, window: int):
        self.n_edges = [int(x) for x in n_edges]
        self.c_edges = [int(x) for x in c_edges]
        self.window = int(window)
        self.kept = [[[] for _ in self.c_edges] for _ in self.n_edges]
        self.records = 0

    @staticmethod
    def bucket(value: int, edges) -> int:
        for i, e in enumerate(edges):
            if value <= e:
                return i
        return len(edges) - 1

    def record(self, n: int, c: int, predicted_ns: int, observed_ns: int) -> None:
        cell = self.kept[self.bucket(n, self.n_edges)][self.bucket(c, self.c_edges)]
        cell.append(max(0, int(observed_ns) - int(predicted_ns)))
        if len(cell) > self.window:
            del cell[0]
        self.records += 1

    @staticmethod
    def nearest_rank(values, percentile_ppm: int) -> int:
        ordered = sorted(values)
        rank = -(-percentile_ppm * len(ordered) // 1_000_000)   # ceil(p * N) in integers
        return ordered[max(rank, 1) - 1]

    def margin(self, n: int, c: int, percentile_ppm: int = 990_000, min_samples: int = 1, floor_ns: int = 0) -> int:
        best = None
        for i in range(self.bucket(n, self.n_edges) + 1):
            for j in range(self.bucket(c, self.c_edges) + 1):
                cell = self.kept[i][j]
                v = self.nearest_rank(cell, percentile_ppm) if len(cell) >= max(min_samples, 1) else int(floor_ns)
                best = v if best is None else max(best, v)
        return best

    def reset(self) -> None:
        """Forget every residual (a new cost table makes the old residuals meaningless)."""
        self.kept = [[[] for _ in self.c_edges] for _ in self.n_edges]

    def exceeds(self, n: int, c: int, configured_margin_ns: int, percentile_ppm: int = 990_000, min_samples: int = 1) -> bool:
        return self.margin(n, c, percentile_ppm, min_samples, 0) > configured_margin_ns

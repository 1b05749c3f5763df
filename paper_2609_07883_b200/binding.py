"""ctypes binding of ``include/sw.h`` — argument marshalling only.

Functions carry the C names (``sw_create``, ``sw_kv_append``, ``sw_mixed_attn_run``, ``sw_cost_probe``,
``sw_choose_chunk`` ...).  torch is used for device memory and streams only; every step of the path runs in
the library's kernels.  Loading fails loudly if ``libsloweave.so`` has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import numpy as np

import os

# SLOWEAVE_LIB names another build of the same library to load instead of the default file: the sanitizer run of the
# CPU tests loads ``libsloweave_asan.so`` (``build.build_sanitized()``) this way.
_LIB_PATH = Path(os.environ.get("SLOWEAVE_LIB") or Path(__file__).resolve().parent / "libsloweave.so")
if not _LIB_PATH.exists():
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_07883_b200.build` "
                      "(there is no CPU or library fallback)")
_lib = C.CDLL(str(_LIB_PATH))

SW_OK, SW_ERR_INVALID_ARG, SW_ERR_OUT_OF_RANGE, SW_ERR_UNSUPPORTED = 0, 1, 2, 3
SW_ERR_WORKSPACE, SW_ERR_CUDA, SW_ERR_DEVICE_TIMEOUT, SW_ERR_NOT_MONOTONE = 4, 5, 6, 7
SW_F_NO_PREFILL, SW_F_NO_DECODE, SW_F_DECODE_INFEASIBLE, SW_F_CAPPED = 1, 2, 4, 8
INT64_MAX = (1 << 63) - 1


class sw_layout(C.Structure):
    _fields_ = [("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_size", C.c_int32), ("num_pages", C.c_int64), ("sm_scale", C.c_float)]


class sw_batch(C.Structure):
    _fields_ = [("prefix_len", C.c_int32), ("chunk_len", C.c_int32), ("prefill_pages", C.c_void_p),
                ("num_prefill_pages", C.c_int32), ("num_decode", C.c_int32), ("decode_kv_len", C.c_void_p),
                ("decode_page_indptr", C.c_void_p), ("decode_pages", C.c_void_p), ("num_chunks", C.c_int32),
                ("chunk_prefix_lens", C.c_void_p), ("chunk_lens", C.c_void_p), ("chunk_page_indptr", C.c_void_p)]


def _chunk_fields(batch):
    """(num_chunks, three HOST pointers, keepalive) of a batch's chunk arrays; zeros for a single-chunk batch."""
    if getattr(batch, "chunk_lens", None) is None:
        return 0, None, None, None, []
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in
            (batch.chunk_prefix_lens, batch.chunk_lens, batch.chunk_page_indptr)]
    return len(arrs[1]), arrs[0].ctypes.data, arrs[1].ctypes.data, arrs[2].ctypes.data, arrs


class sw_chooser_params(C.Structure):
    _fields_ = [("margin_abs_ns", C.c_int64), ("margin_ppm", C.c_int32), ("c_max", C.c_int32),
                ("chunk_quantum", C.c_int32)]


class sw_choice(C.Structure):
    _fields_ = [("chunk", C.c_int32), ("flags", C.c_int32), ("budget_ns", C.c_int64), ("predicted_ns", C.c_int64),
                ("queries", C.c_int32)]


class sw_telemetry_totals(C.Structure):
    _fields_ = [("records", C.c_int64), ("fallbacks", C.c_int64), ("deadline_misses", C.c_int64),
                ("max_residual_ns", C.c_int64)]


EXPORTS = ["sw_workspace_bytes", "sw_create", "sw_destroy", "sw_kv_append", "sw_mixed_attn_run", "sw_mixed_iteration_run",
           "sw_mixed_iteration_host", "sw_cost_probe", "sw_cost_probe_iteration", "sw_check_status", "sw_cost_table_create",
           "sw_cost_table_destroy", "sw_cost_table_lookup", "sw_choose_chunk", "sw_choose_chunks", "sw_last_error",
           "sw_decode_attn_static", "sw_selftest_wait_timeout", "sw_telemetry_create", "sw_telemetry_destroy",
           "sw_telemetry_record", "sw_telemetry_margin", "sw_telemetry_exceeds", "sw_telemetry_get_totals",
           "sw_telemetry_reset"]

_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64
_lib.sw_workspace_bytes.restype = C.c_size_t
_lib.sw_workspace_bytes.argtypes = [C.POINTER(sw_layout), _i32, _i32, _i64]
_lib.sw_create.argtypes = [C.POINTER(sw_layout), C.c_int, _vp, C.c_size_t, _i32, _i32, _i64, C.POINTER(_vp)]
_lib.sw_destroy.argtypes = [_vp]
_lib.sw_destroy.restype = None
_lib.sw_kv_append.argtypes = [_vp, _vp, C.POINTER(sw_batch), _vp, _vp, _vp]
_lib.sw_mixed_attn_run.argtypes = [_vp, _vp, C.POINTER(sw_batch), _vp, _vp, _vp, _vp]
_lib.sw_mixed_iteration_run.argtypes = [_vp, _vp, C.POINTER(sw_batch), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sw_mixed_iteration_host.argtypes = [_vp, _vp, C.POINTER(sw_batch), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.sw_cost_probe.argtypes = [_vp, C.POINTER(_vp), _i32, C.POINTER(sw_batch), _vp, _vp, _i32, _i32,
                               C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), _vp]
_lib.sw_cost_probe_iteration.argtypes = [_vp, C.POINTER(_vp), _i32, C.POINTER(sw_batch), _vp, _vp, _vp, _vp, _i32, _i32,
                                         C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), _vp]
_lib.sw_decode_attn_static.argtypes = [C.POINTER(sw_layout), C.c_int, _vp, C.POINTER(sw_batch), _vp, _vp, _vp, _vp]
_lib.sw_selftest_wait_timeout.argtypes = [_vp, _i64, _vp]
_lib.sw_check_status.argtypes = [_vp, _vp, C.POINTER(_i32), C.POINTER(_i32)]
_lib.sw_cost_table_create.argtypes = [C.POINTER(_i32), _i32, C.POINTER(_i64), _i32, C.POINTER(_i32), _i32,
                                      C.POINTER(_i32), _i32, C.POINTER(_i64), C.c_int, C.c_int, C.POINTER(_vp)]
_lib.sw_cost_table_destroy.argtypes = [_vp]
_lib.sw_choose_chunks.argtypes = [_vp, C.POINTER(sw_chooser_params), _i64, C.POINTER(_i64), _i32, _i64, C.POINTER(_i32),
                                  C.POINTER(_i32), _i32, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(sw_choice)]
_lib.sw_telemetry_create.argtypes = [C.POINTER(_i32), _i32, C.POINTER(_i32), _i32, _i32, C.POINTER(_vp)]
_lib.sw_telemetry_destroy.argtypes = [_vp]
_lib.sw_telemetry_destroy.restype = None
_lib.sw_telemetry_record.argtypes = [_vp, _i32, _i32, _i64, _i64, _i64, _i32]
_lib.sw_telemetry_margin.argtypes = [_vp, _i32, _i32, _i32, _i32, _i64, C.POINTER(_i64)]
_lib.sw_telemetry_exceeds.argtypes = [_vp, _i32, _i32, _i32, _i32, _i64, C.POINTER(_i32)]
_lib.sw_telemetry_reset.argtypes = [_vp]
_lib.sw_telemetry_get_totals.argtypes = [_vp, C.POINTER(sw_telemetry_totals)]
_lib.sw_cost_table_destroy.restype = None
_lib.sw_cost_table_lookup.argtypes = [_vp, _i64, _i64, _i64, _i64, C.POINTER(_i64)]
_lib.sw_choose_chunk.argtypes = [_vp, C.POINTER(sw_chooser_params), _i64, C.POINTER(_i64), _i32, _i64, _i32, _i32,
                                 C.POINTER(sw_choice)]
_lib.sw_last_error.restype = C.c_char_p


class SwError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status}: {_lib.sw_last_error().decode()}")


def _check(status: int, where: str) -> None:
    if status != SW_OK:
        raise SwError(status, where)


def sw_last_error() -> str:
    return _lib.sw_last_error().decode()


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor / numpy array, or None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_handle(stream) -> int:
    import torch

    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def make_layout(shape, num_pages: int, sm_scale: float = 0.0) -> sw_layout:
    return sw_layout(shape.num_q_heads, shape.num_kv_heads, shape.head_dim, shape.page_size, int(num_pages),
                     float(sm_scale))


# ---------------------------------------------------------------------------------------------------------------
# device path
# ---------------------------------------------------------------------------------------------------------------
def sw_workspace_bytes(layout: sw_layout, max_chunk: int, max_decode: int, max_pages: int) -> int:
    return int(_lib.sw_workspace_bytes(C.byref(layout), max_chunk, max_decode, max_pages))


class Context:
    """Owns the workspace tensor and the opaque ``sw_ctx``."""

    def __init__(self, shape, num_pages: int, max_chunk: int, max_decode: int, max_pages: int, device: int = 0,
                 sm_scale: float = 0.0):
        import torch

        self.shape = shape
        self.layout = make_layout(shape, num_pages, sm_scale)
        self.device = torch.device("cuda", device)
        nbytes = sw_workspace_bytes(self.layout, max_chunk, max_decode, max_pages)
        if nbytes == 0:
            raise SwError(SW_ERR_UNSUPPORTED, "sw_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        handle = _vp()
        _check(_lib.sw_create(C.byref(self.layout), device, self.workspace.data_ptr(), nbytes, max_chunk, max_decode,
                              max_pages, C.byref(handle)), "sw_create")
        self.handle = handle

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.sw_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


class DeviceBatch:
    """A ``workloads.MixedBatch`` with its index arrays on the device and the matching ``sw_batch`` struct."""

    def __init__(self, batch, device):
        import torch

        self.host = batch
        to = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.prefill_pages = to(batch.prefill_pages)
        self.decode_kv_len = to(batch.decode_kv_len)
        self.decode_page_indptr = to(batch.decode_page_indptr)
        self.decode_pages = to(batch.decode_pages)
        nch, cp, cl, ci, self._chunk_keep = _chunk_fields(batch)
        self.struct = sw_batch(batch.prefix_len, batch.chunk_len, self.prefill_pages.data_ptr(),
                               int(self.prefill_pages.numel()), batch.num_decode, self.decode_kv_len.data_ptr(),
                               self.decode_page_indptr.data_ptr(), self.decode_pages.data_ptr(), nch, cp, cl, ci)


def host_batch_struct(batch):
    """``sw_batch`` whose pointers are HOST pointers (for sw_mixed_iteration_host); returns (struct, keepalive)."""
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in
            (batch.prefill_pages, batch.decode_kv_len, batch.decode_page_indptr, batch.decode_pages)]
    nch, cp, cl, ci, keep = _chunk_fields(batch)
    s = sw_batch(batch.prefix_len, batch.chunk_len, arrs[0].ctypes.data, int(arrs[0].shape[0]), batch.num_decode,
                 arrs[1].ctypes.data, arrs[2].ctypes.data, arrs[3].ctypes.data, nch, cp, cl, ci)
    return s, arrs + keep


def sw_kv_append(ctx: Context, kv_pool, batch: DeviceBatch, k_new, v_new, stream=None) -> None:
    _check(_lib.sw_kv_append(ctx.handle, _ptr(kv_pool), C.byref(batch.struct), _ptr(k_new), _ptr(v_new),
                             _stream_handle(stream)), "sw_kv_append")


def sw_mixed_attn_run(ctx: Context, kv_pool, batch: DeviceBatch, q, out, lse=None, stream=None) -> None:
    _check(_lib.sw_mixed_attn_run(ctx.handle, _ptr(kv_pool), C.byref(batch.struct), _ptr(q), _ptr(out), _ptr(lse),
                                  _stream_handle(stream)), "sw_mixed_attn_run")


def sw_mixed_iteration_run(ctx: Context, kv_pool, batch: DeviceBatch, k_new, v_new, q, out, lse=None, stream=None) -> None:
    _check(_lib.sw_mixed_iteration_run(ctx.handle, _ptr(kv_pool), C.byref(batch.struct), _ptr(k_new), _ptr(v_new), _ptr(q),
                                       _ptr(out), _ptr(lse), _stream_handle(stream)), "sw_mixed_iteration_run")


def sw_mixed_iteration_host(ctx: Context, kv_pool, host_struct: sw_batch, h_q, h_k_new, h_v_new, h_out, h_lse=None,
                            stream=None) -> None:
    _check(_lib.sw_mixed_iteration_host(ctx.handle, _ptr(kv_pool), C.byref(host_struct), _ptr(h_q), _ptr(h_k_new),
                                        _ptr(h_v_new), _ptr(h_out), _ptr(h_lse), _stream_handle(stream)),
           "sw_mixed_iteration_host")


def sw_cost_probe_iteration(ctx: Context, kv_pools, batch: DeviceBatch, k_new, v_new, q, out, warmup: int = 3,
                            reps: int = 30, stream=None):
    """As ``sw_cost_probe`` with the KV append fused into every timed launch."""
    layers = len(kv_pools)
    arr = (_vp * layers)(*[_ptr(p) for p in kv_pools])
    p50, p99 = _i64(0), _i64(0)
    samples = np.zeros(reps, dtype=np.int64)
    _check(_lib.sw_cost_probe_iteration(ctx.handle, arr, layers, C.byref(batch.struct), _ptr(k_new), _ptr(v_new), _ptr(q),
                                        _ptr(out), warmup, reps, C.byref(p50), C.byref(p99),
                                        samples.ctypes.data_as(C.POINTER(_i64)), _stream_handle(stream)),
           "sw_cost_probe_iteration")
    return int(p50.value), int(p99.value), samples


def sw_cost_probe(ctx: Context, kv_pools, batch: DeviceBatch, q, out, warmup: int = 3, reps: int = 30, stream=None):
    """Returns (p50_ns, p99_ns, samples_ns ndarray) per iteration over the ``kv_pools`` layer stack."""
    layers = len(kv_pools)
    arr = (_vp * layers)(*[_ptr(p) for p in kv_pools])
    p50, p99 = _i64(0), _i64(0)
    samples = np.zeros(reps, dtype=np.int64)
    _check(_lib.sw_cost_probe(ctx.handle, arr, layers, C.byref(batch.struct), _ptr(q), _ptr(out), warmup, reps,
                              C.byref(p50), C.byref(p99), samples.ctypes.data_as(C.POINTER(_i64)),
                              _stream_handle(stream)), "sw_cost_probe")
    return int(p50.value), int(p99.value), samples


def sw_check_status(ctx: Context, stream=None, raise_on_error: bool = True):
    code, detail = _i32(0), _i32(0)
    st = _lib.sw_check_status(ctx.handle, _stream_handle(stream), C.byref(code), C.byref(detail))
    if st != SW_OK and raise_on_error:
        raise SwError(st, "sw_check_status")
    return int(code.value), int(detail.value)


SW_STATIC_MAX_DECODE = 128


def sw_selftest_wait_timeout(ctx: Context, budget_cycles: int = 200_000, stream=None) -> None:
    """Launch the bounded-wait self-test: a wait that cannot succeed gives up and reports SW_ERR_DEVICE_TIMEOUT."""
    _check(_lib.sw_selftest_wait_timeout(ctx.handle, int(budget_cycles), _stream_handle(stream)), "sw_selftest_wait_timeout")


def sw_decode_attn_static(layout: sw_layout, device: int, kv_pool, batch: DeviceBatch, q, out, lse=None, stream=None) -> None:
    """Decode-only attention that allocates nothing: its scratch is a fixed array inside the library image, so it
    needs neither a Context nor a workspace (for callers that may not call cudaMalloc)."""
    _check(_lib.sw_decode_attn_static(C.byref(layout), device, _ptr(kv_pool), C.byref(batch.struct), _ptr(q), _ptr(out),
                                      _ptr(lse), _stream_handle(stream)), "sw_decode_attn_static")




# ---------------------------------------------------------------------------------------------------------------
# controller (host only)
# ---------------------------------------------------------------------------------------------------------------
class CostTable:
    def __init__(self, n_grid, ctx_grid, prefix_grid, chunk_grid, cost_ns, make_monotone: bool = True,
                 interp: bool = False):
        ng = np.ascontiguousarray(n_grid, dtype=np.int32)
        cg = np.ascontiguousarray(ctx_grid, dtype=np.int64)
        pg = np.ascontiguousarray(prefix_grid, dtype=np.int32)
        kg = np.ascontiguousarray(chunk_grid, dtype=np.int32)
        cost = np.ascontiguousarray(cost_ns, dtype=np.int64).reshape(-1)
        if cost.shape[0] != len(ng) * len(cg) * len(pg) * len(kg):
            raise ValueError("cost_ns has the wrong number of entries")
        handle = _vp()
        pi32 = lambda a: a.ctypes.data_as(C.POINTER(_i32))
        pi64 = lambda a: a.ctypes.data_as(C.POINTER(_i64))
        _check(_lib.sw_cost_table_create(pi32(ng), len(ng), pi64(cg), len(cg), pi32(pg), len(pg), pi32(kg), len(kg),
                                         pi64(cost), int(make_monotone), int(interp), C.byref(handle)),
               "sw_cost_table_create")
        self.handle = handle

    def lookup(self, n: int, ctx: int, prefix: int, c: int) -> int:
        out = _i64(0)
        _check(_lib.sw_cost_table_lookup(self.handle, n, ctx, prefix, c, C.byref(out)), "sw_cost_table_lookup")
        return int(out.value)

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.sw_cost_table_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


SW_MAX_CHUNKS = 8


def sw_choose_chunks(table, now_ns: int, deadlines_ns, total_ctx: int, prefix_lens, remaining_prefill, c_max: int = 4096,
                     chunk_quantum: int = 1, margin_abs_ns: int = 0, margin_ppm: int = 0):
    """First fit over the pending requests (oldest first).  Returns (list of admitted chunk lengths, sw_choice)."""
    dl = np.ascontiguousarray(deadlines_ns, dtype=np.int64)
    pre = np.ascontiguousarray(prefix_lens, dtype=np.int32)
    rem = np.ascontiguousarray(remaining_prefill, dtype=np.int32)
    if pre.shape != rem.shape:
        raise ValueError("prefix_lens and remaining_prefill differ in length")
    params = sw_chooser_params(margin_abs_ns, margin_ppm, c_max, chunk_quantum)
    chunks = np.zeros(SW_MAX_CHUNKS, dtype=np.int32)
    count = _i32(0)
    out = sw_choice()
    pi32 = lambda a: a.ctypes.data_as(C.POINTER(_i32))
    _check(_lib.sw_choose_chunks(table.handle if table is not None else None, C.byref(params), now_ns,
                                 dl.ctypes.data_as(C.POINTER(_i64)), len(dl), total_ctx, pi32(pre), pi32(rem), len(rem),
                                 pi32(chunks), C.byref(count), C.byref(out)), "sw_choose_chunks")
    return [int(x) for x in chunks[:count.value]], out


class Telemetry:
    """Residual table of the online feedback loop (``sw_telemetry_*``)."""

    def __init__(self, n_edges, c_edges, window: int = 256):
        ne = np.ascontiguousarray(n_edges, dtype=np.int32)
        ce = np.ascontiguousarray(c_edges, dtype=np.int32)
        handle = _vp()
        _check(_lib.sw_telemetry_create(ne.ctypes.data_as(C.POINTER(_i32)), len(ne), ce.ctypes.data_as(C.POINTER(_i32)),
                                        len(ce), window, C.byref(handle)), "sw_telemetry_create")
        self.handle = handle

    def record(self, n: int, c: int, predicted_ns: int, observed_ns: int, slack_ns: int = 0, fallback: bool = False) -> None:
        _check(_lib.sw_telemetry_record(self.handle, n, c, predicted_ns, observed_ns, slack_ns, int(fallback)),
               "sw_telemetry_record")

    def margin(self, n: int, c: int, percentile_ppm: int = 990_000, min_samples: int = 1, floor_ns: int = 0) -> int:
        out = _i64(0)
        _check(_lib.sw_telemetry_margin(self.handle, n, c, percentile_ppm, min_samples, floor_ns, C.byref(out)),
               "sw_telemetry_margin")
        return int(out.value)

    def exceeds(self, n: int, c: int, configured_margin_ns: int, percentile_ppm: int = 990_000, min_samples: int = 1) -> bool:
        out = _i32(0)
        _check(_lib.sw_telemetry_exceeds(self.handle, n, c, percentile_ppm, min_samples, configured_margin_ns,
                                         C.byref(out)), "sw_telemetry_exceeds")
        return bool(out.value)

    def reset(self) -> None:
        _check(_lib.sw_telemetry_reset(self.handle), "sw_telemetry_reset")

    def totals(self) -> dict:
        t = sw_telemetry_totals()
        _check(_lib.sw_telemetry_get_totals(self.handle, C.byref(t)), "sw_telemetry_get_totals")
        return {k: int(getattr(t, k)) for k, _ in t._fields_}

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.sw_telemetry_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


def sw_choose_chunk(table: CostTable | None, now_ns: int, deadlines_ns, total_ctx: int, prefix_len: int,
                    remaining_prefill: int, c_max: int = 4096, chunk_quantum: int = 1, margin_abs_ns: int = 0,
                    margin_ppm: int = 0) -> sw_choice:
    dl = np.ascontiguousarray(deadlines_ns, dtype=np.int64)
    params = sw_chooser_params(margin_abs_ns, margin_ppm, c_max, chunk_quantum)
    out = sw_choice()
    _check(_lib.sw_choose_chunk(table.handle if table is not None else None, C.byref(params), now_ns,
                                dl.ctypes.data_as(C.POINTER(_i64)), len(dl), total_ctx, prefix_len, remaining_prefill,
                                C.byref(out)), "sw_choose_chunk")
    return out

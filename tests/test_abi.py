"""The C-ABI library loads without a GPU and exports every symbol the public header declares."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_07883_b200 import build

    return build.build()


def declared_functions():
    text = (ROOT / "include" / "sw.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sw_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for must in ("sw_mixed_attn_run", "sw_kv_append", "sw_cost_probe", "sw_choose_chunk"):
        assert must in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(str(lib_path))
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in include/sw.h but not exported"


def test_binding_lists_the_same_functions(lib_path):
    from paper_2609_07883_b200 import binding

    assert sorted(binding.EXPORTS) == declared_functions()
    for name in binding.EXPORTS:
        # handles are wrapped by classes (Context, CostTable, Telemetry); everything else has a function of the same name
        assert hasattr(binding, name) or name.startswith("sw_telemetry_") or name in (
            "sw_create", "sw_destroy", "sw_cost_table_create", "sw_cost_table_destroy", "sw_cost_table_lookup")
    assert all(hasattr(binding, cls) for cls in ("Context", "CostTable", "Telemetry"))


def test_host_side_argument_errors_without_a_gpu(lib_path):
    from paper_2609_07883_b200 import binding as B
    from paper_2609_07883_b200 import workloads as W

    assert B.sw_workspace_bytes(B.make_layout(W.LLAMA, 1024), 512, 64, 4096) > 0
    assert B.sw_workspace_bytes(B.make_layout(W.AttnShape(32, 8, 96), 1024), 512, 64, 4096) == 0   # head_dim
    assert B.sw_workspace_bytes(B.make_layout(W.AttnShape(32, 8, 128, page_size=32), 1024), 1, 1, 1) == 0
    assert B.sw_workspace_bytes(B.make_layout(W.AttnShape(48, 4, 128), 1024), 1, 1, 1) == 0        # group 12
    with pytest.raises(B.SwError) as e:
        B.CostTable([1, 2], [10], [0], [0, 16], [5, 4, 6, 7], make_monotone=False)
    assert e.value.status == B.SW_ERR_NOT_MONOTONE
    with pytest.raises(B.SwError) as e:
        B.CostTable([2, 1], [10], [0], [0, 16], [1, 2, 3, 4])
    assert e.value.status == B.SW_ERR_INVALID_ARG


def test_static_entry_point_refuses_bad_arguments_before_any_cuda_call(lib_path):
    """Host-side refusals of sw_decode_attn_static: they come before the first CUDA call, so they can be checked here."""
    import ctypes as C

    from paper_2609_07883_b200 import binding as B
    from paper_2609_07883_b200 import workloads as W

    fake = 0x1000  # aligned, never dereferenced: every call below is refused on its arguments
    lay = B.make_layout(W.AttnShape(8, 2, 128), 64)
    one = B.sw_batch(0, 0, None, 0, 1, fake, fake, fake, 0, None, None, None)
    call = lambda layout, device, batch: B._lib.sw_decode_attn_static(C.byref(layout), device, fake, C.byref(batch), fake,
                                                                      fake, None, None)
    assert call(lay, -1, one) == B.SW_ERR_INVALID_ARG and "out of range" in B.sw_last_error()
    assert call(lay, 64, one) == B.SW_ERR_INVALID_ARG
    too_many = B.sw_batch(0, 0, None, 0, B.SW_STATIC_MAX_DECODE + 1, fake, fake, fake, 0, None, None, None)
    assert call(lay, 0, too_many) == B.SW_ERR_WORKSPACE and "static limit" in B.sw_last_error()
    chunked = B.sw_batch(0, 16, fake, 1, 1, fake, fake, fake, 0, None, None, None)
    assert call(lay, 0, chunked) == B.SW_ERR_UNSUPPORTED
    assert call(B.make_layout(W.AttnShape(32, 16, 128), 64), 0, one) == B.SW_ERR_WORKSPACE   # more than 8 KV heads

"""CPU-side checks of the C ABI: the library loads, exports what the header declares, and validates
arguments on the host before touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def resq():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2412_14363_b200 as m
    return m


def _declared_functions(header="resq.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(resq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(resq):
    names = _declared_functions()
    assert {"resq_pack_weights", "resq_project_quantize", "resq_mixed_gemm", "resq_linear"} <= set(names)
    for n in names:
        assert hasattr(resq.lib, n), n
    assert sorted(resq.EXPORTS) == names


def test_pack_projected_host_validation(resq):
    L = resq.lib
    import ctypes
    d = resq.layer_desc(512, 64, 64)
    fake = 1 << 20
    need = L.resq_pack_projected_workspace_bytes(ctypes.byref(d))
    assert need == 64 * 512 * 4
    assert L.resq_pack_projected_workspace_bytes(ctypes.byref(resq.layer_desc(500, 64, 64))) == 0
    assert L.resq_pack_weights_projected(ctypes.byref(d), fake, None, fake, fake, fake, fake, None, fake, need, None) == resq.ERR_NULL
    assert L.resq_pack_weights_projected(ctypes.byref(d), fake, fake, fake, fake, fake, fake, None, fake, need - 1, None) == resq.ERR_WORKSPACE
    assert L.resq_pack_weights_projected(ctypes.byref(d), fake + 2, fake, fake, fake, fake, fake, None, fake, need, None) == resq.ERR_ALIGN


def test_project_host_validation(resq):
    L = resq.lib
    fake = 1 << 20
    assert L.resq_project_workspace_bytes() == 74 * 256 * 256 * 4
    assert L.resq_project(fake, fake, 4, 1001, fake, None, 0, None) == resq.ERR_SHAPE
    assert L.resq_project(fake, None, 4, 1024, fake, None, 0, None) == resq.ERR_NULL
    assert L.resq_project(fake, fake, 4, 1024, fake, fake + 8, 1 << 30, None) == resq.ERR_ALIGN


def test_every_header_is_covered():
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["resq.h", "resq_kv.h"]


def test_library_exports_every_kv_symbol(resq):
    from paper_2412_14363_b200 import kv
    names = _declared_functions("resq_kv.h")
    assert "resq_attention_decode" in names and "resq_kv_append" in names
    for n in names:
        assert hasattr(resq.lib, n), n
    assert sorted(kv.KV_EXPORTS) == names


def test_kv_host_validation(resq):
    """Geometry, NULL and alignment checks of the attention-block entry points (nothing is launched)."""
    import ctypes
    from paper_2412_14363_b200 import kv
    L = resq.lib
    assert L.resq_kv_cache_bytes(2, 8, 128, 64) == 2 * 8 * 2 * 5632
    assert L.resq_kv_cache_bytes(2, 8, 64, 64) == 2 * 8 * 2 * 3328    # d_head = 64: every code array halved
    assert L.resq_kv_block_bytes(128) == 5632 and L.resq_kv_block_bytes(64) == 3328 and L.resq_kv_block_bytes(96) == 0
    assert L.resq_kv_cache_bytes(2, 8, 96, 64) == 0 and L.resq_kv_cache_bytes(2, 8, 128, 48) == 0
    assert L.resq_kv_cache_bytes(0, 8, 128, 64) == 0
    assert L.resq_attention_workspace_bytes(4, 32, 8, 128) > 0
    assert L.resq_attention_workspace_bytes(4, 30, 8, 128) == 0      # not a multiple of the KV heads
    assert L.resq_attention_workspace_bytes(4, 72, 8, 128) == 0      # more than 8 query heads per KV head
    fake = 1 << 20
    c = kv.KvCacheStruct(2, 8, 128, 64, fake)
    assert L.resq_uc_quantize(fake, 96, fake, fake, None) == resq.ERR_SHAPE
    assert L.resq_uc_quantize(None, 128, fake, fake, None) == resq.ERR_NULL
    assert L.resq_query_project(fake, 5, 128, fake, fake + 4, fake, None) == resq.ERR_ALIGN
    assert L.resq_query_project(fake, -1, 128, fake, fake, fake, None) == resq.ERR_SHAPE
    assert L.resq_kv_append(None, fake, fake, 1, fake, fake, fake, fake, None) == resq.ERR_NULL
    assert L.resq_kv_append(ctypes.byref(c), fake, None, 1, fake, fake, fake, fake, None) == resq.ERR_NULL
    bad = kv.KvCacheStruct(2, 8, 128, 40, fake)
    assert L.resq_kv_append(ctypes.byref(bad), fake, fake, 1, fake, fake, fake, fake, None) == resq.ERR_SHAPE
    assert L.resq_attention_decode(ctypes.byref(c), fake, 32, fake, fake, fake, 16, None) == resq.ERR_WORKSPACE
    assert L.resq_attention_decode(ctypes.byref(c), fake, 12, fake, fake, fake, 1 << 30, None) == resq.ERR_SHAPE
    assert "index" in resq.status_string(kv.ERR_INDEX)


def test_status_strings(resq):
    assert resq.status_string(0) == "ok"
    assert "workspace" in resq.status_string(resq.ERR_WORKSPACE)
    assert resq.status_string(99) == "unknown status"


def test_size_queries(resq):
    d = resq.layer_desc(4096, 4096, 512)
    assert resq.lib.resq_w8_bytes(ctypes.byref(d)) == 4096 * 512
    assert resq.lib.resq_w4_bytes(ctypes.byref(d)) == 4096 * 3584 // 2
    assert resq.lib.resq_w4_i8_bytes(ctypes.byref(d)) == 4096 * 3584
    assert resq.lib.resq_scale_bytes(ctypes.byref(d)) == 4096 * 4
    d16 = resq.layer_desc(4096, 4096, 512, resq.SCALE_FP16)
    assert resq.lib.resq_scale_bytes(ctypes.byref(d16)) == 4096 * 2
    # one block of the 8B-shaped model packs to 122.9 MB (0.5625 bytes per weight)
    total = 0
    for K, N in ((4096, 4096), (4096, 1024), (4096, 1024), (4096, 4096), (4096, 14336), (4096, 14336), (14336, 4096)):
        dd = resq.layer_desc(K, N, K // 8)
        total += resq.lib.resq_w8_bytes(ctypes.byref(dd)) + resq.lib.resq_w4_bytes(ctypes.byref(dd))
    assert abs(total / 1e6 - 122.7) < 0.5
    assert resq.resq_workspace_bytes(d, 4096, False, True) > 4096 * 3584
    assert resq.resq_workspace_bytes(d, 4096, True, True) > resq.resq_workspace_bytes(d, 4096, False, True)
    assert resq.resq_workspace_bytes(resq.layer_desc(4096, 4096, 500), 16, False, True) == 0


def test_host_validation_happens_before_any_launch(resq):
    """Bad arguments are rejected with their status code; none of these calls needs a device."""
    L = resq.lib
    good = resq.layer_desc(512, 512, 64)
    fake = 0x10000  # 16-byte aligned, never dereferenced on the host
    ws = resq.WeightsStruct(fake, fake, fake, fake, None)
    W = ctypes.byref(ws)
    # shape rules
    for K, N, r in ((512, 512, -32), (512, 512, 512), (512, 512, 48), (500, 512, 64), (512, 508, 64), (0, 8, 0)):
        bad = resq.layer_desc(K, N, r)
        assert L.resq_mixed_gemm(ctypes.byref(bad), 16, fake, fake, None, fake, fake, W, fake, 0, None, None, fake, 1 << 30, None) == resq.ERR_SHAPE
        assert L.resq_pack_weights(ctypes.byref(bad), fake, fake, fake, fake, fake, None, None) == resq.ERR_SHAPE
    assert L.resq_mixed_gemm(ctypes.byref(good), 0, fake, fake, None, fake, fake, W, fake, 0, None, None, fake, 1 << 30, None) == resq.ERR_SHAPE
    assert L.resq_mixed_gemm(ctypes.byref(good), 16, fake, fake, None, fake, fake, W, fake, 7, None, None, fake, 1 << 30, None) == resq.ERR_SHAPE
    assert L.resq_project_quantize(fake, None, 16, 512, 60, fake, fake, fake, fake, None, None, 0, None) == resq.ERR_SHAPE
    # the Hadamard path: a width with no construction here, a misaligned input, a missing output
    assert L.resq_hadamard_quantize(fake, 4, 1000, 0, None, fake, fake, fake, None, None) == resq.ERR_SHAPE
    assert L.resq_hadamard_quantize(fake + 2, 4, 1024, 0, None, fake, fake, fake, None, None) == resq.ERR_ALIGN
    assert L.resq_hadamard_quantize(fake, 4, 1024, 128, None, fake, fake, fake, None, None) == resq.ERR_NULL
    # null pointers
    assert L.resq_mixed_gemm(None, 16, fake, fake, None, fake, fake, W, fake, 0, None, None, fake, 1 << 30, None) == resq.ERR_NULL
    assert L.resq_mixed_gemm(ctypes.byref(good), 16, None, fake, None, fake, fake, W, fake, 0, None, None, fake, 1 << 30, None) == resq.ERR_NULL
    assert L.resq_mixed_gemm(ctypes.byref(good), 16, fake, fake, None, fake, fake, W, fake, 0, fake, None, fake, 1 << 30, None) == resq.ERR_NULL
    assert L.resq_linear(ctypes.byref(good), 16, None, None, W, fake, 0, fake, 1 << 30, None) == resq.ERR_NULL
    assert L.resq_pack_weights(ctypes.byref(good), None, fake, fake, fake, fake, None, None) == resq.ERR_NULL
    assert L.resq_project_quantize(fake, None, 16, 512, 64, fake, None, fake, fake, None, None, 0, None) == resq.ERR_NULL
    wnull = resq.WeightsStruct(fake, None, fake, fake, None)
    assert L.resq_linear(ctypes.byref(good), 16, fake, None, ctypes.byref(wnull), fake, 0, fake, 1 << 30, None) == resq.ERR_NULL
    # alignment
    assert L.resq_mixed_gemm(ctypes.byref(good), 16, fake + 4, fake, None, fake, fake, W, fake, 0, None, None, fake, 1 << 30, None) == resq.ERR_ALIGN
    assert L.resq_linear(ctypes.byref(good), 16, fake, None, W, fake + 8, 0, fake, 1 << 30, None) == resq.ERR_ALIGN
    assert L.resq_project_quantize(fake + 2, None, 16, 512, 64, fake, fake, fake, fake, None, None, 0, None) == resq.ERR_ALIGN
    # workspace
    need = resq.resq_workspace_bytes(good, 64, False, False)
    assert L.resq_mixed_gemm(ctypes.byref(good), 64, fake, fake, None, fake, fake, W, fake, 0, None, None, fake, need - 1, None) == resq.ERR_WORKSPACE
    assert L.resq_mixed_gemm(ctypes.byref(good), 64, fake, fake, None, fake, fake, W, fake, 0, None, None, None, 0, None) == resq.ERR_WORKSPACE
    assert L.resq_linear(ctypes.byref(good), 64, fake, None, W, fake, 0, fake, 16, None) == resq.ERR_WORKSPACE


def test_options_and_error_text(resq):
    """Host-only entry points: an unknown option is refused, the known one toggles, and the CUDA error
    text is a string even when no CUDA error has occurred."""
    assert resq.lib.resq_set_option(12345, 1) == resq.ERR_SHAPE
    assert resq.lib.resq_set_option(resq.OPT_WAIT_LIMIT_US, 0) == resq.ERR_SHAPE      # refused before any device call
    assert resq.lib.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 1) == resq.OK
    assert resq.lib.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 0) == resq.OK
    assert isinstance(resq.lib.resq_last_cuda_error(), bytes)

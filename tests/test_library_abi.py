"""The shared library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2609_33135_b200 import build
    return build.build()


def test_exports_every_declared_symbol(built):
    header = open(os.path.join(ROOT, "include", "mpfa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(mpfa_[a-z0-9_]+)\s*\(", header))
    assert {"mpfa_quantize_qk", "mpfa_quantize_v", "mpfa_prefill", "mpfa_decode"} <= names
    lib = ctypes.CDLL(built)
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_host_only_helpers(built):
    from paper_2609_33135_b200 import binding
    L = binding.lib()
    assert L.mpfa_version() >= 100
    assert L.mpfa_fp4_codes_bytes(1, 2, 130) == 2 * 256 * 64
    assert L.mpfa_fp4_sf_bytes(1, 2, 130) == 2 * 2 * 1024
    assert L.mpfa_delta_s_bytes(1, 4, 130) == 4 * 256 * 2
    assert L.mpfa_v_fp8_bytes(2, 2, 128) == 2 * 2 * 128 * 128
    assert L.mpfa_v_fp4_bytes(2, 3, 130) == 2 * 3 * 2 * (8192 + 1024) and L.mpfa_v_fp4_bytes(1, 0, 5) == 0
    assert L.mpfa_fp4_codes_bytes(0, 1, 1) == 0
    assert L.mpfa_status_string(0) == b"ok" and L.mpfa_status_string(-3) == b"misaligned buffer"
    # layout maps agree with the documented formulas and are bijections
    from layouts import paged_k_offset, paged_v_offset
    seen = set()
    for t in range(128):
        for g in range(8):
            off = L.mpfa_sf_offset(1, 128, 0, 0, t, g)
            assert off == (g // 4) * 512 + (t % 32) * 16 + (t // 32) * 4 + g % 4
            seen.add(off)
    assert seen == set(range(1024))
    assert L.mpfa_sf_offset(3, 300, 1, 2, 257, 5) == ((1 * 3 + 2) * 3 + 2) * 1024 + 512 + 16 + 1
    ks = {L.mpfa_paged_k_offset(t, g, j) for t in range(64) for g in range(8) for j in range(8)}
    assert ks == set(range(4096))
    assert all(L.mpfa_paged_k_offset(t, g, j) == paged_k_offset(t, g, j)
               for t in (0, 7, 8, 63) for g in (0, 5) for j in (0, 3, 7))
    vs = {L.mpfa_paged_v_offset(t, c) for t in range(64) for c in range(128)}
    assert vs == set(range(8192))
    assert all(L.mpfa_paged_v_offset(t, c) == paged_v_offset(t, c) for t in (0, 9, 31, 40, 63) for c in (0, 8, 17, 127))


def test_argument_errors_without_gpu(built):
    """Host-side validation runs before any CUDA call."""
    from paper_2609_33135_b200 import binding
    L = binding.lib()
    st = binding._Stats(0, 0, 0, 0)
    assert L.mpfa_quantize_qk(None, None, 1, 1, 1, 1, 1, 0, ctypes.byref(st), None, None, None, None, 0, None) == -1
    assert L.mpfa_quantize_v(None, 1, 1, 1, 1.0, None, None) == -1
    assert L.mpfa_quantize_v_fp4(None, 1, 1, 1, 1.0, None, None) == -1
    assert L.mpfa_pack_v_bf16(None, 1, 1, 1, None, None) == -1
    assert L.mpfa_prefill(None, None, None, None, None, 1.0, 0, 1.0, None, None, None, None) == -1
    assert L.mpfa_prefill_variant(None, None, None, None, None, 1.0, 0, 1.0, 0, None, None, None, None) == -1
    assert L.mpfa_prefill_variant(None, None, None, None, None, 1.0, 0, 1.0, 5, None, None, None, None) == -1
    assert L.mpfa_prefill_paged(None, None, None, 1, None, None, None, 1.0, 1.0, None, None, None, None) == -1
    assert L.mpfa_decode(None, None, None, 1, None, None, 1.0, 1.0, None, None, None, 0, None, None) == -1
    assert L.mpfa_quantize_kv_paged(None, None, 1, 0, 1, 1, 0, None, 1.0, None, None, None, 0, None) == -1
    assert L.mpfa_append_kv_paged(None, None, 1, 1, 1, 0, None, 1.0, None, None, 1, None, None) == -1


def test_paged_entry_points_validate_shapes_before_any_cuda_call(built):
    """Shape and alignment errors of the paged calls are found on the host (fake but well-aligned addresses,
    nothing is dereferenced)."""
    from paper_2609_33135_b200 import binding
    L = binding.lib()
    a = 1 << 20   # a 1 MiB-aligned fake device address
    st = binding._Stats(a, a, a, a)
    q = binding._Fp4(a, a, 1, 8, 100)
    kv = binding._PagedKV(a, a, a, a, 4, 64, 8, 2)
    args = (ctypes.byref(q), ctypes.byref(kv), ctypes.c_void_p(a), 4, ctypes.c_void_p(a), None, ctypes.byref(st), 1.0, 0.088,
            ctypes.c_void_p(a), None, ctypes.c_void_p(a), None)
    kv_bad_page = binding._PagedKV(a, a, a, a, 4, 32, 8, 2)
    assert L.mpfa_prefill_paged(args[0], ctypes.byref(kv_bad_page), *args[2:]) == -2          # page_size != 64
    kv_bad_heads = binding._PagedKV(a, a, a, a, 4, 64, 6, 2)
    assert L.mpfa_prefill_paged(args[0], ctypes.byref(kv_bad_heads), *args[2:]) == -1         # cache sized for other heads
    kv_bad_group = binding._PagedKV(a, a, a, a, 4, 64, 8, 3)
    assert L.mpfa_prefill_paged(args[0], ctypes.byref(kv_bad_group), *args[2:]) == -2         # H_q % H_kv != 0
    kv_unaligned = binding._PagedKV(a + 8, a, a, a, 4, 64, 8, 2)
    assert L.mpfa_prefill_paged(args[0], ctypes.byref(kv_unaligned), *args[2:]) == -3         # pool not 256-byte aligned
    assert L.mpfa_prefill_paged(*args[:7], 0.0, *args[8:]) == -1                               # v_scale must be positive
    assert L.mpfa_prefill_paged(*args[:3], 0, *args[4:]) == -1                                 # max_pages_per_req

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
    assert L.mpfa_prefill(None, None, None, None, None, 1.0, 0, 1.0, None, None, None, None) == -1

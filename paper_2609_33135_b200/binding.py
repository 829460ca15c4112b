"""ctypes binding of libmpfa.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and the current CUDA stream; every step of the path runs
inside the library's kernels.  There is no fallback: if the shared library is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmpfa.so")

MPFA_SMOOTH = 1
MPFA_STATS_FROZEN = 2
MPFA_DEV_TIMEOUT = 1
MPFA_DEV_BAD_PAGE = 2
MPFA_VARIANT_COMP_ELEMENTWISE = 1
MPFA_VARIANT_PV_BF16 = 2
MPFA_VARIANT_PV_FP4 = 3
HEAD_DIM = 128
PAGE = 64


class MpfaError(RuntimeError):
    pass


class _Stats(ctypes.Structure):
    _fields_ = [("q_mean", ctypes.c_void_p), ("k_mean", ctypes.c_void_p),
                ("q_gscale", ctypes.c_void_p), ("k_gscale", ctypes.c_void_p)]


class _Fp4(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("sf", ctypes.c_void_p),
                ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32)]


class _PagedKV(ctypes.Structure):
    _fields_ = [("k_codes", ctypes.c_void_p), ("k_sf", ctypes.c_void_p), ("v_fp8", ctypes.c_void_p),
                ("delta_s_bf16", ctypes.c_void_p), ("num_pages", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("H_q", ctypes.c_int32), ("H_kv", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libmpfa.so (built by paper_2609_33135_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        _lib = load_library(LIB_PATH)
    return _lib


def load_library(path: str) -> ctypes.CDLL:
    """A build of the library with the C ABI's argument types declared."""
    if True:
        if not os.path.exists(path):
            raise MpfaError(f"{path} not found: build it with `python -m paper_2609_33135_b200.build`")
        L = ctypes.CDLL(path)
        sz, i, f, vp = ctypes.c_size_t, ctypes.c_int, ctypes.c_float, ctypes.c_void_p
        L.mpfa_quantize_workspace_bytes.restype = sz
        L.mpfa_quantize_workspace_bytes.argtypes = [i, i, i]
        L.mpfa_quantize_workspace_min_bytes.restype = sz
        L.mpfa_quantize_workspace_min_bytes.argtypes = [i, i, i]
        L.mpfa_decode_workspace_bytes.restype = sz
        L.mpfa_decode_workspace_bytes.argtypes = [i, i, i, i]
        for name in ("mpfa_fp4_codes_bytes", "mpfa_fp4_sf_bytes", "mpfa_delta_s_bytes", "mpfa_v_fp8_bytes", "mpfa_v_fp4_bytes"):
            getattr(L, name).restype = sz
            getattr(L, name).argtypes = [i, i, i]
        L.mpfa_sf_offset.restype = sz
        L.mpfa_sf_offset.argtypes = [i, i, i, i, i, i]
        L.mpfa_paged_k_offset.restype = sz
        L.mpfa_paged_k_offset.argtypes = [i, i, i]
        L.mpfa_paged_v_offset.restype = sz
        L.mpfa_paged_v_offset.argtypes = [i, i]
        L.mpfa_status_string.restype = ctypes.c_char_p
        L.mpfa_status_string.argtypes = [i]
        L.mpfa_last_cuda_error.restype = i
        L.mpfa_version.restype = i
        L.mpfa_quantize_qk.restype = i
        L.mpfa_quantize_qk.argtypes = [vp, vp, i, i, i, i, i, i, ctypes.POINTER(_Stats), ctypes.POINTER(_Fp4),
                                       ctypes.POINTER(_Fp4), vp, vp, sz, vp]
        L.mpfa_quantize_qk_static.restype = i
        L.mpfa_quantize_qk_static.argtypes = [vp, vp, i, i, i, i, i, i, ctypes.POINTER(_Stats), ctypes.POINTER(_Fp4),
                                              ctypes.POINTER(_Fp4), vp, vp]
        L.mpfa_static_scratch_bytes.restype = sz
        L.mpfa_quantize_v.restype = i
        L.mpfa_quantize_v.argtypes = [vp, i, i, i, f, vp, vp]
        L.mpfa_quantize_v_fp4.restype = i
        L.mpfa_quantize_v_fp4.argtypes = [vp, i, i, i, f, vp, vp]
        L.mpfa_pack_v_bf16.restype = i
        L.mpfa_pack_v_bf16.argtypes = [vp, i, i, i, vp, vp]
        L.mpfa_quantize_kv_paged.restype = i
        L.mpfa_quantize_kv_paged.argtypes = [vp, vp, i, i, i, i, i, ctypes.POINTER(_Stats), f,
                                             ctypes.POINTER(_PagedKV), vp, vp, sz, vp]
        L.mpfa_append_kv_paged.restype = i
        L.mpfa_append_kv_paged.argtypes = [vp, vp, i, i, i, i, ctypes.POINTER(_Stats), f, ctypes.POINTER(_PagedKV), vp, i,
                                           vp, vp]
        L.mpfa_prefill.restype = i
        L.mpfa_prefill.argtypes = [ctypes.POINTER(_Fp4), ctypes.POINTER(_Fp4), vp, vp, ctypes.POINTER(_Stats), f, i,
                                   f, vp, vp, vp, vp]
        L.mpfa_decode.restype = i
        L.mpfa_decode.argtypes = [ctypes.POINTER(_Fp4), ctypes.POINTER(_PagedKV), vp, i, vp, ctypes.POINTER(_Stats),
                                  f, f, vp, vp, vp, sz, vp, vp]
        L.mpfa_prefill_variant.restype = i
        L.mpfa_prefill_variant.argtypes = [ctypes.POINTER(_Fp4), ctypes.POINTER(_Fp4), vp, vp, ctypes.POINTER(_Stats), f, i,
                                           f, i, vp, vp, vp, vp]
        L.mpfa_prefill_paged.restype = i
        L.mpfa_prefill_paged.argtypes = [ctypes.POINTER(_Fp4), ctypes.POINTER(_PagedKV), vp, i, vp, vp,
                                         ctypes.POINTER(_Stats), f, f, vp, vp, vp, vp]
        L.mpfa_set_prefill_arrangement.restype = i
        L.mpfa_set_prefill_arrangement.argtypes = [i]
        L.mpfa_bench_mma_peak.restype = i
        L.mpfa_bench_mma_peak.argtypes = [i, i, i, vp, vp]
        L.mpfa_bench_mma_flops.restype = ctypes.c_double
        L.mpfa_bench_mma_flops.argtypes = [i, i, i]
        return L


def _check(rc: int, what: str) -> None:
    if rc != 0:
        L = lib()
        msg = L.mpfa_status_string(rc).decode()
        raise MpfaError(f"{what}: {msg} (status {rc}, cuda error {L.mpfa_last_cuda_error()})")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _pad128(n: int) -> int:
    return (n + 127) // 128 * 128


def aligned_empty(nbytes: int, device="cuda", align: int = 1024, zero: bool = False) -> torch.Tensor:
    """uint8 device buffer whose data pointer is a multiple of `align` (torch's allocator only
    guarantees 512 bytes; the TMA-fed tiles want 1024)."""
    alloc = torch.zeros if zero else torch.empty
    raw = alloc(nbytes + align, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % align
    return raw[off:off + nbytes]


@dataclass
class Stats:
    """Per-request statistics (device tensors): means [B,H,128] and per-tensor scales [B]."""
    q_mean: torch.Tensor
    k_mean: torch.Tensor
    q_gscale: torch.Tensor
    k_gscale: torch.Tensor

    @staticmethod
    def empty(B: int, H_q: int, H_kv: int, device="cuda") -> "Stats":
        return Stats(torch.zeros(B, H_q, HEAD_DIM, dtype=torch.float32, device=device),
                     torch.zeros(B, H_kv, HEAD_DIM, dtype=torch.float32, device=device),
                     torch.ones(B, dtype=torch.float32, device=device),
                     torch.ones(B, dtype=torch.float32, device=device))

    def c(self) -> _Stats:
        return _Stats(self.q_mean.data_ptr(), self.k_mean.data_ptr(), self.q_gscale.data_ptr(),
                      self.k_gscale.data_ptr())

    def request(self, b: int) -> "Stats":
        """View of one request's statistics (B = 1 slices)."""
        return Stats(self.q_mean[b:b + 1], self.k_mean[b:b + 1], self.q_gscale[b:b + 1], self.k_gscale[b:b + 1])


@dataclass
class Fp4Tensor:
    """NVFP4 tensor in the library's tile layout (device uint8 buffers)."""
    codes: torch.Tensor
    sf: torch.Tensor
    B: int
    H: int
    N: int

    @staticmethod
    def empty(B: int, H: int, N: int, device="cuda") -> "Fp4Tensor":
        L = lib()
        return Fp4Tensor(aligned_empty(L.mpfa_fp4_codes_bytes(B, H, N), device),
                         aligned_empty(L.mpfa_fp4_sf_bytes(B, H, N), device), B, H, N)

    def c(self) -> _Fp4:
        return _Fp4(self.codes.data_ptr(), self.sf.data_ptr(), self.B, self.H, self.N)


@dataclass
class PagedKV:
    """Paged low-bit KV cache (device uint8 / bf16 pools)."""
    k_codes: torch.Tensor
    k_sf: torch.Tensor
    v_fp8: torch.Tensor
    delta: Optional[torch.Tensor]
    num_pages: int
    H_q: int
    H_kv: int

    @staticmethod
    def empty(num_pages: int, H_q: int, H_kv: int, with_delta: bool = True, device="cuda") -> "PagedKV":
        return PagedKV(torch.zeros(num_pages, H_kv, 4096, dtype=torch.uint8, device=device),
                       torch.zeros(num_pages, H_kv, 512, dtype=torch.uint8, device=device),
                       torch.zeros(num_pages, H_kv, 8192, dtype=torch.uint8, device=device),
                       torch.zeros(num_pages, H_q, PAGE, dtype=torch.bfloat16, device=device) if with_delta else None,
                       num_pages, H_q, H_kv)

    def c(self) -> _PagedKV:
        return _PagedKV(self.k_codes.data_ptr(), self.k_sf.data_ptr(), self.v_fp8.data_ptr(),
                        None if self.delta is None else self.delta.data_ptr(), self.num_pages, PAGE,
                        self.H_q, self.H_kv)


def quantize_workspace(B: int, H_q: int, H_kv: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(256, lib().mpfa_quantize_workspace_bytes(B, H_q, H_kv)), dtype=torch.uint8, device=device)


def mpfa_quantize_qk(q: Optional[torch.Tensor], k: Optional[torch.Tensor], flags: int, stats: Stats,
                     q_out: Optional[Fp4Tensor], k_out: Optional[Fp4Tensor], delta: Optional[torch.Tensor],
                     workspace: Optional[torch.Tensor], H_q: Optional[int] = None, H_kv: Optional[int] = None) -> None:
    """q [B,N_q,H_q,128], k [B,N_kv,H_kv,128] bf16 device tensors (either may be None)."""
    ref = q if q is not None else k
    B = ref.shape[0]
    N_q = q.shape[1] if q is not None else 0
    N_kv = k.shape[1] if k is not None else 0
    H_q = q.shape[2] if q is not None else (H_q if H_q is not None else stats.q_mean.shape[1])
    H_kv = k.shape[2] if k is not None else (H_kv if H_kv is not None else stats.k_mean.shape[1])
    for t in (q, k):
        assert t is None or (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape[3] == HEAD_DIM)
    sc = stats.c()
    qc = q_out.c() if q_out is not None else None
    kc = k_out.c() if k_out is not None else None
    rc = lib().mpfa_quantize_qk(_ptr(q), _ptr(k), B, N_q, N_kv, H_q, H_kv, flags, ctypes.byref(sc),
                                ctypes.byref(qc) if qc is not None else None,
                                ctypes.byref(kc) if kc is not None else None, _ptr(delta), _ptr(workspace),
                                0 if workspace is None else workspace.numel(), _stream())
    _check(rc, "mpfa_quantize_qk")


def mpfa_quantize_qk_static(q: Optional[torch.Tensor], k: Optional[torch.Tensor], flags: int, stats: Stats,
                            q_out: Optional[Fp4Tensor], k_out: Optional[Fp4Tensor],
                            delta: Optional[torch.Tensor]) -> None:
    """mpfa_quantize_qk without a workspace argument: for callers that may not allocate device
    memory.  The library's own fixed scratch buffer is used; shapes that need more than
    mpfa_static_scratch_bytes() raise MpfaError("workspace too small").  This wrapper itself
    allocates nothing on the device.  Calls overlapping on the GPU share that buffer and race."""
    ref = q if q is not None else k
    B = ref.shape[0]
    N_q = q.shape[1] if q is not None else 0
    N_kv = k.shape[1] if k is not None else 0
    H_q = q.shape[2] if q is not None else stats.q_mean.shape[1]
    H_kv = k.shape[2] if k is not None else stats.k_mean.shape[1]
    sc = stats.c()
    qc = q_out.c() if q_out is not None else None
    kc = k_out.c() if k_out is not None else None
    rc = lib().mpfa_quantize_qk_static(_ptr(q), _ptr(k), B, N_q, N_kv, H_q, H_kv, flags, ctypes.byref(sc),
                                       ctypes.byref(qc) if qc is not None else None,
                                       ctypes.byref(kc) if kc is not None else None, _ptr(delta), _stream())
    _check(rc, "mpfa_quantize_qk_static")


def mpfa_quantize_v(v: torch.Tensor, v_scale: float, out: torch.Tensor) -> None:
    assert v.is_cuda and v.dtype == torch.bfloat16 and v.is_contiguous()
    B, N, H, _ = v.shape
    _check(lib().mpfa_quantize_v(_ptr(v), B, N, H, v_scale, _ptr(out), _stream()), "mpfa_quantize_v")


def mpfa_quantize_kv_paged(k: torch.Tensor, v: torch.Tensor, first_token: int, H_q: int, flags: int, stats: Stats,
                           v_scale: float, kv: PagedKV, page_table_row: torch.Tensor,
                           workspace: Optional[torch.Tensor]) -> None:
    """k, v [N_tokens, H_kv, 128] bf16 of ONE request; stats are that request's B = 1 slices."""
    assert k.is_cuda and k.dtype == torch.bfloat16 and k.is_contiguous() and v.is_contiguous()
    assert page_table_row.dtype == torch.int32 and page_table_row.is_cuda
    N, H_kv, _ = k.shape
    sc, kc = stats.c(), kv.c()
    rc = lib().mpfa_quantize_kv_paged(_ptr(k), _ptr(v), N, first_token, H_q, H_kv, flags, ctypes.byref(sc), v_scale,
                                      ctypes.byref(kc), _ptr(page_table_row), _ptr(workspace),
                                      0 if workspace is None else workspace.numel(), _stream())
    _check(rc, "mpfa_quantize_kv_paged")


def mpfa_append_kv_paged(k: torch.Tensor, v: torch.Tensor, H_q: int, flags: int, stats: Stats, v_scale: float,
                         kv: PagedKV, page_table: torch.Tensor, positions: torch.Tensor) -> None:
    """k, v: [B, 1, H_kv, 128] bf16; one new token per request at positions[b]."""
    assert k.dtype == torch.bfloat16 and k.is_contiguous() and v.is_contiguous() and k.shape == v.shape
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and positions.dtype == torch.int32
    B, one, H_kv, _ = k.shape
    assert one == 1
    sc, kc = stats.c(), kv.c()
    rc = lib().mpfa_append_kv_paged(_ptr(k), _ptr(v), B, H_q, H_kv, flags, ctypes.byref(sc), v_scale, ctypes.byref(kc),
                                    _ptr(page_table), page_table.shape[1], _ptr(positions), _stream())
    _check(rc, "mpfa_append_kv_paged")


def mpfa_prefill(q: Fp4Tensor, k: Fp4Tensor, v_fp8: torch.Tensor, delta: Optional[torch.Tensor], stats: Stats,
                 v_scale: float, causal: bool, softmax_scale: float, out: torch.Tensor,
                 out_f32: Optional[torch.Tensor], device_status: torch.Tensor) -> None:
    sc, qc, kc = stats.c(), q.c(), k.c()
    rc = lib().mpfa_prefill(ctypes.byref(qc), ctypes.byref(kc), _ptr(v_fp8), _ptr(delta), ctypes.byref(sc), v_scale,
                            int(causal), softmax_scale, _ptr(out), _ptr(out_f32), _ptr(device_status), _stream())
    _check(rc, "mpfa_prefill")


def mpfa_prefill_variant(q: Fp4Tensor, k: Fp4Tensor, v_fp8: torch.Tensor, delta: Optional[torch.Tensor], stats: Stats,
                         v_scale: float, causal: bool, softmax_scale: float, variant: int, out: torch.Tensor,
                         out_f32: Optional[torch.Tensor], device_status: torch.Tensor) -> None:
    sc, qc, kc = stats.c(), q.c(), k.c()
    rc = lib().mpfa_prefill_variant(ctypes.byref(qc), ctypes.byref(kc), _ptr(v_fp8), _ptr(delta), ctypes.byref(sc), v_scale,
                                    int(causal), softmax_scale, int(variant), _ptr(out), _ptr(out_f32),
                                    _ptr(device_status), _stream())
    _check(rc, "mpfa_prefill_variant")


def decode_workspace(B: int, H_q: int, H_kv: int, max_pages: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(256, lib().mpfa_decode_workspace_bytes(B, H_q, H_kv, max_pages)), dtype=torch.uint8,
                       device=device)


def mpfa_decode(q: Fp4Tensor, kv: PagedKV, page_table: torch.Tensor, seq_lens: torch.Tensor, stats: Stats,
                v_scale: float, softmax_scale: float, out: torch.Tensor, out_f32: Optional[torch.Tensor],
                workspace: torch.Tensor, device_status: torch.Tensor) -> None:
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and seq_lens.dtype == torch.int32
    sc, qc, kc = stats.c(), q.c(), kv.c()
    rc = lib().mpfa_decode(ctypes.byref(qc), ctypes.byref(kc), _ptr(page_table), page_table.shape[1], _ptr(seq_lens),
                           ctypes.byref(sc), v_scale, softmax_scale, _ptr(out), _ptr(out_f32), _ptr(workspace),
                           workspace.numel(), _ptr(device_status), _stream())
    _check(rc, "mpfa_decode")


def mpfa_prefill_paged(q: Fp4Tensor, kv: PagedKV, page_table: torch.Tensor, seq_lens: torch.Tensor, stats: Stats,
                       v_scale: float, softmax_scale: float, out: torch.Tensor, out_f32: Optional[torch.Tensor],
                       device_status: torch.Tensor, q_lens: Optional[torch.Tensor] = None) -> None:
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and seq_lens.dtype == torch.int32
    assert q_lens is None or q_lens.dtype == torch.int32
    sc, qc, kc = stats.c(), q.c(), kv.c()
    rc = lib().mpfa_prefill_paged(ctypes.byref(qc), ctypes.byref(kc), _ptr(page_table), page_table.shape[1],
                                  _ptr(seq_lens), _ptr(q_lens), ctypes.byref(sc), v_scale, softmax_scale, _ptr(out),
                                  _ptr(out_f32), _ptr(device_status), _stream())
    _check(rc, "mpfa_prefill_paged")


# ---------------------------------------------------------------------------------------
# Convenience wrappers: allocate the outputs with torch, then make the calls above.
# ---------------------------------------------------------------------------------------
@dataclass
class Stage1:
    q: Fp4Tensor
    k: Fp4Tensor
    v_fp8: torch.Tensor
    delta: Optional[torch.Tensor]
    stats: Stats
    v_scale: float


def stage1(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, smooth: bool = True, v_scale: float = 1.0,
           workspace: Optional[torch.Tensor] = None, out: Optional[Stage1] = None) -> Stage1:
    """Algorithm 1 lines 1-5 on device tensors q [B,N_q,H_q,128], k, v [B,N_kv,H_kv,128]."""
    B, N_q, H_q, _ = q.shape
    N_kv, H_kv = k.shape[1], k.shape[2]
    dev = q.device
    if out is None:
        L = lib()
        out = Stage1(Fp4Tensor.empty(B, H_q, N_q, dev), Fp4Tensor.empty(B, H_kv, N_kv, dev),
                     aligned_empty(L.mpfa_v_fp8_bytes(B, H_kv, N_kv), dev),
                     aligned_empty(L.mpfa_delta_s_bytes(B, H_q, N_kv), dev).view(torch.bfloat16).view(
                         B, H_q, _pad128(N_kv)) if smooth else None,
                     Stats.empty(B, H_q, H_kv, dev), v_scale)
    if workspace is None:
        workspace = quantize_workspace(B, H_q, H_kv, dev)
    mpfa_quantize_qk(q, k, MPFA_SMOOTH if smooth else 0, out.stats, out.q, out.k, out.delta, workspace)
    mpfa_quantize_v(v, v_scale, out.v_fp8)
    return out


def prefill(s1: Stage1, causal: bool, softmax_scale: float, want_f32: bool = False,
            out: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    """Algorithm 1 lines 6-20.  Returns (out_bf16 [B,N_q,H_q,128], out_f32 or None, status int32[1])."""
    B, H_q, N_q = s1.q.B, s1.q.H, s1.q.N
    dev = s1.q.codes.device
    if out is None:
        out = torch.empty(B, N_q, H_q, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    o32 = torch.empty(B, N_q, H_q, HEAD_DIM, dtype=torch.float32, device=dev) if want_f32 else None
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    mpfa_prefill(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, s1.v_scale, causal, softmax_scale, out, o32, status)
    return out, o32, status


def mpfa_bench_mma_peak(kind: int, n_cols: int, iters: int, status: torch.Tensor) -> float:
    """Enqueue the tensor-core rate probe; returns the FLOPs the whole grid issues (one CTA per SM)."""
    _check(lib().mpfa_bench_mma_peak(kind, n_cols, iters, _ptr(status), _stream()), "mpfa_bench_mma_peak")
    n_sm = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    return float(lib().mpfa_bench_mma_flops(kind, n_cols, iters)) * n_sm


def mpfa_set_prefill_arrangement(arrangement: int) -> None:
    """0 (default): one query tile per CTA; 1: two query tiles per CTA.  Same arithmetic row by row."""
    _check(lib().mpfa_set_prefill_arrangement(arrangement), "mpfa_set_prefill_arrangement")


def mpfa_pack_v_bf16(v: torch.Tensor) -> torch.Tensor:
    """V [B,N,H,128] bf16 -> the BF16 tile tensor [B,H,N_pad,128] the MPFA_VARIANT_PV_BF16 prefill reads."""
    assert v.is_cuda and v.dtype == torch.bfloat16 and v.is_contiguous()
    B, N, H, _ = v.shape
    out = aligned_empty(2 * lib().mpfa_v_fp8_bytes(B, H, N), v.device).view(torch.bfloat16).view(B, H, _pad128(N), HEAD_DIM)
    _check(lib().mpfa_pack_v_bf16(_ptr(v), B, N, H, _ptr(out), _stream()), "mpfa_pack_v_bf16")
    return out


def mpfa_quantize_v_fp4(v: torch.Tensor, v_gscale: float) -> torch.Tensor:
    """V [B,N,H,128] bf16 -> the FP4 operand (codes of all tiles, then block scales) the MPFA_VARIANT_PV_FP4 prefill reads."""
    assert v.is_cuda and v.dtype == torch.bfloat16 and v.is_contiguous()
    B, N, H, _ = v.shape
    out = aligned_empty(lib().mpfa_v_fp4_bytes(B, H, N), v.device)
    _check(lib().mpfa_quantize_v_fp4(_ptr(v), B, N, H, v_gscale, _ptr(out), _stream()), "mpfa_quantize_v_fp4")
    return out

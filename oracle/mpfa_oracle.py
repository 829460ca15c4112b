"""ctypes front end of the CPU oracle (oracle/mpfa_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's cpu_baseline / reference arm.  The CUDA library and its Python
binding never import this module, and this module never imports them.

All arrays are numpy; BF16 tensors travel as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mpfa_oracle.c")
_LIB = os.path.join(_HERE, "libmpfa_oracle.so")

D = 128
NBLK = 8
BLOCK_KV = 128      # KV block of the main loop (Algorithm 1; 128 x 128 score tile, Section 3.2)
DECODE_SPLIT = 1024  # decode partition: 8 x 128 tokens (Section 5.3)

CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", *CFLAGS, "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.mpfa_oracle_bf16_to_f32.restype = ctypes.c_float
        _lib.mpfa_oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.mpfa_oracle_f32_to_bf16.restype = ctypes.c_uint16
        _lib.mpfa_oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.mpfa_oracle_e4m3_decode.restype = ctypes.c_float
        _lib.mpfa_oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        _lib.mpfa_oracle_e4m3_encode.restype = ctypes.c_uint8
        _lib.mpfa_oracle_e4m3_encode.argtypes = [ctypes.c_float]
        _lib.mpfa_oracle_e2m1_decode.restype = ctypes.c_float
        _lib.mpfa_oracle_e2m1_decode.argtypes = [ctypes.c_uint8]
        _lib.mpfa_oracle_e2m1_encode.restype = ctypes.c_uint8
        _lib.mpfa_oracle_e2m1_encode.argtypes = [ctypes.c_float]
    return _lib


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def bf16_bits(t) -> np.ndarray:
    """torch BF16 tensor (CPU) -> numpy uint16 bit patterns (no copy when contiguous)."""
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.uint16).numpy()


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


# --- scalar format helpers (used by the pins) --------------------------------
def e4m3_encode(x: float) -> int:
    return int(lib().mpfa_oracle_e4m3_encode(ctypes.c_float(x)))


def e4m3_decode(c: int) -> float:
    return float(lib().mpfa_oracle_e4m3_decode(ctypes.c_uint8(c)))


def e2m1_encode(x: float) -> int:
    return int(lib().mpfa_oracle_e2m1_encode(ctypes.c_float(x)))


def e2m1_decode(c: int) -> float:
    return float(lib().mpfa_oracle_e2m1_decode(ctypes.c_uint8(c)))


def f32_to_bf16(x: float) -> int:
    return int(lib().mpfa_oracle_f32_to_bf16(ctypes.c_float(x)))


# --- stage 1 -------------------------------------------------------------------
def means(x: np.ndarray) -> np.ndarray:
    """x: uint16 [B,N,H,128] -> FP32 [B,H,128] (Eq. 7)."""
    B, N, H, d = x.shape
    assert d == D
    out = np.empty((B, H, D), np.float32)
    lib().mpfa_oracle_means(_p(x), B, N, H, _p(out))
    return out


def colsum_fixed(x: np.ndarray) -> np.ndarray:
    B, N, H, d = x.shape
    out = np.empty((B, H, D), np.int64)
    lib().mpfa_oracle_colsum_fixed(_p(x), B, N, H, _p(out))
    return out


def tensor_scale(x: np.ndarray, mean: np.ndarray) -> np.ndarray:
    B, N, H, d = x.shape
    out = np.empty((B,), np.float32)
    lib().mpfa_oracle_tensor_scale(_p(x), _p(_c(mean, np.float32)), B, N, H, _p(out))
    return out


def quantize_nvfp4(x: np.ndarray, mean: np.ndarray, d: np.ndarray):
    """-> codes uint8 [B,H,N,64], sf uint8 [B,H,N,8] (Eq. 1)."""
    B, N, H, _ = x.shape
    codes = np.empty((B, H, N, D // 2), np.uint8)
    sf = np.empty((B, H, N, NBLK), np.uint8)
    lib().mpfa_oracle_quantize_nvfp4(_p(x), _p(_c(mean, np.float32)), _p(_c(d, np.float32)), B, N, H,
                                     _p(codes), _p(sf))
    return codes, sf


def delta_s(k: np.ndarray, q_mean, k_mean, dq, dk, Hq: int) -> np.ndarray:
    """-> BF16 bits [B,Hq,N] (Eq. 9, in MMA units)."""
    B, N, Hkv, _ = k.shape
    out = np.empty((B, Hq, N), np.uint16)
    lib().mpfa_oracle_delta_s(_p(k), _p(_c(q_mean, np.float32)), _p(_c(k_mean, np.float32)),
                              _p(_c(dq, np.float32)), _p(_c(dk, np.float32)), B, N, Hq, Hkv, _p(out))
    return out


def quantize_v(v: np.ndarray, v_scale: float = 1.0) -> np.ndarray:
    """-> uint8 [B,H,N,128] E4M3 codes."""
    B, N, H, _ = v.shape
    out = np.empty((B, H, N, D), np.uint8)
    lib().mpfa_oracle_quantize_v(_p(v), B, N, H, ctypes.c_float(v_scale), _p(out))
    return out


@dataclass
class Quantized:
    """Everything stage 1 hands to stage 2 (logical row-major arrays)."""
    q_codes: np.ndarray   # [B,Hq,Nq,64]
    q_sf: np.ndarray      # [B,Hq,Nq,8]
    k_codes: np.ndarray   # [B,Hkv,Nkv,64]
    k_sf: np.ndarray      # [B,Hkv,Nkv,8]
    v_codes: np.ndarray   # [B,Hkv,Nkv,128]
    delta: Optional[np.ndarray]  # BF16 bits [B,Hq,Nkv] or None
    q_mean: np.ndarray    # [B,Hq,128]
    k_mean: np.ndarray    # [B,Hkv,128]
    dq: np.ndarray        # [B]
    dk: np.ndarray        # [B]
    v_scale: float


def stage1(q: np.ndarray, k: np.ndarray, v: np.ndarray, smooth: bool = True, v_scale: float = 1.0,
           frozen: Optional[Quantized] = None) -> Quantized:
    """Algorithm 1 lines 1-5.  smooth=False is the paper's "direct" variant
    (means forced to zero, no compensation vector).  With `frozen`, the means
    and tensor scales of an earlier call are reused (decode, Section 6)."""
    B, Nq, Hq, _ = q.shape
    Hkv = k.shape[2]
    if frozen is not None:
        qm, km, dq, dk = frozen.q_mean, frozen.k_mean, frozen.dq, frozen.dk
    else:
        qm = means(q) if smooth else np.zeros((B, Hq, D), np.float32)
        km = means(k) if smooth else np.zeros((B, Hkv, D), np.float32)
        dq = tensor_scale(q, qm)
        dk = tensor_scale(k, km)
    qc, qs = quantize_nvfp4(q, qm, dq)
    kc, ks = quantize_nvfp4(k, km, dk)
    dl = delta_s(k, qm, km, dq, dk, Hq) if smooth else None
    vc = quantize_v(v, v_scale)
    return Quantized(qc, qs, kc, ks, vc, dl, qm, km, dq, dk, v_scale)


# --- stage 2 -------------------------------------------------------------------
def prefill_rows(z: Quantized, rows: np.ndarray, softmax_scale: float, causal: bool,
                 block_kv: int = BLOCK_KV, reverse: bool = True, p_fp8: bool = True,
                 use_delta: bool = True, elementwise: bool = False):
    """QK4PV8 prefill outputs for rows [n,3]=(b,hq,i): (FP32 [n,128], BF16 bits [n,128]).
    elementwise=True: the ablation placement of Section 7.4 (Delta_S added to the finished FP32 score)."""
    rows = _c(rows, np.int32)
    B, Hq, Nq, _ = z.q_codes.shape
    Hkv, Nkv = z.k_codes.shape[1], z.k_codes.shape[2]
    n = rows.shape[0]
    o32 = np.empty((n, D), np.float32)
    o16 = np.empty((n, D), np.uint16)
    delta = z.delta if use_delta else None
    fn = lib().mpfa_oracle_prefill_rows_elementwise if elementwise else lib().mpfa_oracle_prefill_rows
    fn(_p(z.q_codes), _p(z.q_sf), _p(z.k_codes), _p(z.k_sf), _p(z.v_codes), _p(delta), _p(_c(z.dq, np.float32)),
       _p(_c(z.dk, np.float32)), ctypes.c_float(z.v_scale), ctypes.c_float(softmax_scale), int(causal), B, Nq, Nkv, Hq,
       Hkv, block_kv, int(reverse), int(p_fp8), _p(rows), n, _p(o32), _p(o16))
    return o32, o16


def all_rows(B: int, Hq: int, Nq: int) -> np.ndarray:
    b, h, i = np.meshgrid(np.arange(B), np.arange(Hq), np.arange(Nq), indexing="ij")
    return np.stack([b.ravel(), h.ravel(), i.ravel()], axis=1).astype(np.int32)


def decode(q_codes, q_sf, k_codes, k_sf, v_codes, delta, dq, dk, v_scale, softmax_scale, seq_lens,
           block_kv: int = BLOCK_KV, split: int = DECODE_SPLIT, reverse: bool = True, p_fp8: bool = True):
    """QK4PV8 decode: q [B,Hq,64]/[B,Hq,8], K/V/delta logical [B,Hkv,Lmax,...] -> (FP32, BF16 bits) [B,Hq,128]."""
    B, Hq, _ = q_codes.shape
    Hkv, Lmax = k_codes.shape[1], k_codes.shape[2]
    o32 = np.empty((B, Hq, D), np.float32)
    o16 = np.empty((B, Hq, D), np.uint16)
    lib().mpfa_oracle_decode(_p(_c(q_codes, np.uint8)), _p(_c(q_sf, np.uint8)), _p(_c(k_codes, np.uint8)),
                             _p(_c(k_sf, np.uint8)), _p(_c(v_codes, np.uint8)),
                             _p(None if delta is None else _c(delta, np.uint16)),
                             _p(_c(dq, np.float32)), _p(_c(dk, np.float32)), ctypes.c_float(v_scale),
                             ctypes.c_float(softmax_scale), _p(_c(seq_lens, np.int32)), B, Lmax, Hq, Hkv,
                             block_kv, split, int(reverse), int(p_fp8), _p(o32), _p(o16))
    return o32, o16


def mainloop_identity(q, k, v, n_vis, softmax_scale, block_kv=BLOCK_KV, reverse=True):
    """The main loop with identity quantizers: q [n,128], k/v [Nkv,128] FP32 -> (out [n,128], row sums [n])."""
    q, k, v = _c(q, np.float32), _c(k, np.float32), _c(v, np.float32)
    n_vis = _c(n_vis, np.int32)
    n = q.shape[0]
    out = np.empty((n, D), np.float32)
    rs = np.empty((n,), np.float32)
    lib().mpfa_oracle_mainloop_identity(_p(q), _p(k), _p(v), _p(n_vis), n, k.shape[0],
                                        ctypes.c_float(softmax_scale), block_kv, int(reverse), _p(out), _p(rs))
    return out, rs


def exact_rows(q, k, v, rows, softmax_scale: float, causal: bool) -> np.ndarray:
    """FP64 softmax attention (Eq. 2) on the unquantized BF16 inputs for rows [n,3]."""
    rows = _c(rows, np.int32)
    B, Nq, Hq, _ = q.shape
    Nkv, Hkv = k.shape[1], k.shape[2]
    out = np.empty((rows.shape[0], D), np.float64)
    lib().mpfa_oracle_exact_rows(_p(q), _p(k), _p(v), ctypes.c_float(softmax_scale), int(causal), B, Nq, Nkv,
                                 Hq, Hkv, _p(rows), rows.shape[0], _p(out))
    return out


def logits_rows(z: Quantized, rows, use_delta=True) -> np.ndarray:
    rows = _c(rows, np.int32)
    B, Hq, Nq, _ = z.q_codes.shape
    Hkv, Nkv = z.k_codes.shape[1], z.k_codes.shape[2]
    out = np.empty((rows.shape[0], Nkv), np.float32)
    lib().mpfa_oracle_logits_rows(_p(z.q_codes), _p(z.q_sf), _p(z.k_codes), _p(z.k_sf),
                                  _p(z.delta if use_delta else None), Nq, Nkv, Hq, Hkv, _p(rows),
                                  rows.shape[0], _p(out))
    return out


def phat_rows(z: Quantized, rows, softmax_scale: float, causal: bool, block_kv: int = BLOCK_KV,
              reverse: bool = True, use_delta: bool = True, want_q: bool = False, flip_key: int = -1, flip_dir: int = 0):
    """Inspection: E4M3 codes of P-hat per visible key [n,Nkv] and the final (m, l) [n,2] of rows [n,3].
    want_q: also the FP32 values 448 P that were encoded [n,Nkv] and the rows' outputs [n,128] (v_scale 1).
    flip_key >= 0: that key's code is moved by flip_dir steps before it is used (what-if for one P-hat)."""
    rows = _c(rows, np.int32)
    B, Hq, Nq, _ = z.q_codes.shape
    Hkv, Nkv = z.k_codes.shape[1], z.k_codes.shape[2]
    codes = np.empty((rows.shape[0], Nkv), np.uint8)
    ml = np.empty((rows.shape[0], 2), np.float32)
    q = np.empty((rows.shape[0], Nkv), np.float32) if want_q else None
    o = np.empty((rows.shape[0], D), np.float32) if want_q else None
    lib().mpfa_oracle_phat_rows(_p(z.q_codes), _p(z.q_sf), _p(z.k_codes), _p(z.k_sf), _p(z.v_codes),
                                _p(z.delta if use_delta else None), _p(_c(z.dq, np.float32)),
                                _p(_c(z.dk, np.float32)), ctypes.c_float(softmax_scale), int(causal), Nq, Nkv, Hq,
                                Hkv, block_kv, int(reverse), _p(rows), rows.shape[0], _p(codes), _p(ml), _p(q), _p(o),
                                int(flip_key), int(flip_dir))
    return (codes, ml, q, o) if want_q else (codes, ml)


def prefill_rows_pv_bf16(z: Quantized, v_bits: np.ndarray, rows, softmax_scale: float, causal: bool,
                         block_kv: int = BLOCK_KV, use_delta: bool = True):
    """Precision-assignment variant of Section 3.1: NVFP4 logits as in the method, P rounded to BF16, V = the BF16
    input [B,Nkv,Hkv,128] (uint16 bits), FP32 accumulation.  -> (FP32 [n,128], BF16 bits [n,128])."""
    rows = _c(rows, np.int32)
    B, Hq, Nq, _ = z.q_codes.shape
    Hkv, Nkv = z.k_codes.shape[1], z.k_codes.shape[2]
    n = rows.shape[0]
    o32 = np.empty((n, D), np.float32)
    o16 = np.empty((n, D), np.uint16)
    lib().mpfa_oracle_prefill_rows_pv_bf16(_p(z.q_codes), _p(z.q_sf), _p(z.k_codes), _p(z.k_sf), _p(_c(v_bits, np.uint16)),
                                           _p(z.delta if use_delta else None), _p(_c(z.dq, np.float32)),
                                           _p(_c(z.dk, np.float32)), ctypes.c_float(softmax_scale), int(causal), Nq, Nkv,
                                           Hq, Hkv, block_kv, _p(rows), n, _p(o32), _p(o16))
    return o32, o16


def quantize_v_fp4(v: np.ndarray, d: float):
    """V for the NVFP4 + NVFP4 assignment (Section 3.1): 16-token blocks along the key axis, tensor scale d.
    -> (codes uint8 [B,H,128,NB,8], sf uint8 [B,H,128,NB]), NB = ceil(N/16)."""
    B, N, H, _ = v.shape
    NB = (N + 15) // 16
    codes = np.empty((B, H, D, NB, 8), np.uint8)
    sf = np.empty((B, H, D, NB), np.uint8)
    lib().mpfa_oracle_quantize_v_fp4(_p(v), B, N, H, ctypes.c_float(d), _p(codes), _p(sf))
    return codes, sf


def prefill_rows_pv_fp4(z: Quantized, v_codes: np.ndarray, v_sf: np.ndarray, v_gscale: float, rows, softmax_scale: float,
                        causal: bool, block_kv: int = BLOCK_KV, use_delta: bool = True, want_codes: bool = False,
                        flip_key: int = -1, flip_dir: int = 0, flip_blk: int = -1, flip_blk_dir: int = 0):
    """Precision-assignment variant of Section 3.1: NVFP4 logits as in the method, P and V as NVFP4 operands of the
    second MMA.  -> (FP32 [n,128], BF16 bits [n,128]) and, with want_codes, the E2M1 codes [n,Nkv] and E4M3 block
    scales [n,ceil(Nkv/16)] of P, the FP32 values [n,Nkv] the codes were made from and the FP32 block maxima
    [n,ceil(Nkv/16)] the scales were made from.  flip_*: inspection switches (one decision moved by that many code steps)."""
    rows = _c(rows, np.int32)
    B, Hq, Nq, _ = z.q_codes.shape
    Hkv, Nkv = z.k_codes.shape[1], z.k_codes.shape[2]
    n = rows.shape[0]
    o32 = np.empty((n, D), np.float32)
    o16 = np.empty((n, D), np.uint16)
    pc = np.empty((n, Nkv), np.uint8) if want_codes else None
    ps = np.empty((n, (Nkv + 15) // 16), np.uint8) if want_codes else None
    y = np.empty((n, Nkv), np.float32) if want_codes else None
    am = np.empty((n, (Nkv + 15) // 16), np.float32) if want_codes else None
    lib().mpfa_oracle_prefill_rows_pv_fp4(_p(z.q_codes), _p(z.q_sf), _p(z.k_codes), _p(z.k_sf), _p(_c(v_codes, np.uint8)),
                                          _p(_c(v_sf, np.uint8)), _p(z.delta if use_delta else None),
                                          _p(_c(z.dq, np.float32)), _p(_c(z.dk, np.float32)), ctypes.c_float(v_gscale),
                                          ctypes.c_float(softmax_scale), int(causal), Nq, Nkv, Hq, Hkv, block_kv, _p(rows), n,
                                          _p(o32), _p(o16), _p(pc), _p(ps), _p(y), _p(am), int(flip_key), int(flip_dir),
                                          int(flip_blk), int(flip_blk_dir))
    return (o32, o16, pc, ps, y, am) if want_codes else (o32, o16)

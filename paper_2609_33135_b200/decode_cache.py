"""Host-side driver for the paged decode path: builds the low-bit KV cache of a
DecodeWorkload by pushing every request through the library's cache-write call, freezes the
query statistics, quantizes the decode-step query and issues mpfa_decode.  All arithmetic is
in the library's kernels; this module only sequences calls and owns the device buffers."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch

from . import binding as B_
from .workloads import DecodeWorkload


@dataclass
class DecodeState:
    w: DecodeWorkload
    kv: B_.PagedKV
    stats: B_.Stats
    q4: B_.Fp4Tensor
    page_table: torch.Tensor
    seq_lens: torch.Tensor
    workspace: torch.Tensor
    out: torch.Tensor
    out_f32: Optional[torch.Tensor]
    status: torch.Tensor
    v_scale: float
    softmax_scale: float


def build_cache(w: DecodeWorkload, device="cuda", smooth: bool = True, v_scale: float = 1.0,
                kv_device: str = "cpu", want_f32: bool = True) -> DecodeState:
    """kv_device: where each request's BF16 K/V are drawn ("cpu": same tensors the oracle tests
    use; a CUDA device: drawn in place for the full-size benchmark)."""
    flags = B_.MPFA_SMOOTH if smooth else 0
    stats = B_.Stats.empty(w.B, w.H_q, w.H_kv, device)
    kv = B_.PagedKV.empty(w.num_pages, w.H_q, w.H_kv, with_delta=smooth, device=device)
    ws = B_.quantize_workspace(w.B, w.H_q, w.H_kv, device)
    table = w.page_table.to(device)
    # frozen query statistics from the sample tokens (Section 6: statistics come from prefill)
    qs = w.q_sample.to(device)
    scratch = B_.Fp4Tensor.empty(w.B, w.H_q, qs.shape[1], device)
    B_.mpfa_quantize_qk(qs, None, flags, stats, scratch, None, None, ws)
    for b in range(w.B):
        k, v = w.kv_for_request(b, kv_device)
        k, v = k[0].to(device), v[0].to(device)
        B_.mpfa_quantize_kv_paged(k, v, 0, w.H_q, flags, stats.request(b), v_scale, kv, table[b], ws)
        del k, v
    q4 = B_.Fp4Tensor.empty(w.B, w.H_q, 1, device)
    B_.mpfa_quantize_qk(w.q_new.to(device), None, flags | B_.MPFA_STATS_FROZEN, stats, q4, None, None, None)
    return DecodeState(w, kv, stats, q4, table, w.seq_lens.to(device),
                       B_.decode_workspace(w.B, w.H_q, w.H_kv, table.shape[1], device),
                       torch.empty(w.B, w.H_q, 128, dtype=torch.bfloat16, device=device),
                       torch.empty(w.B, w.H_q, 128, dtype=torch.float32, device=device) if want_f32 else None,
                       torch.zeros(1, dtype=torch.int32, device=device), v_scale, w.softmax_scale)


def decode_step(s: DecodeState) -> torch.Tensor:
    B_.mpfa_decode(s.q4, s.kv, s.page_table, s.seq_lens, s.stats, s.v_scale, s.softmax_scale, s.out, s.out_f32,
                   s.workspace, s.status)
    return s.out

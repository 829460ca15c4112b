"""Canary words around every buffer the library writes: outputs, quantized tensors, statistics, workspaces and the
paged pools are carved out of one arena filled with a pattern, with guard bands before and after each of them; after
stage 1, prefill (both arrangements, all variants), the cache writes and decode, every guard byte must still hold
the pattern.  Ragged lengths, so that tile tails and pad rows are exercised; the results are also checked against
runs on ordinary allocations, so the carving itself is known to be harmless."""
import os

import numpy as np
import pytest
import torch

from paper_2609_33135_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5
SUITE_ARRANGEMENT = int(os.environ.get("MPFA_TEST_ARRANGEMENT", "0"))   # what the rest of the suite runs on


class Arena:
    def __init__(self, nbytes: int):
        self.raw = torch.full((nbytes + 2048,), PATTERN, dtype=torch.uint8, device="cuda")
        self.base = (-self.raw.data_ptr()) % 1024
        self.pos = self.base + GUARD
        self.live = []

    def take(self, nbytes: int) -> torch.Tensor:
        start = self.pos
        assert start + nbytes + GUARD <= self.raw.numel(), "arena too small"
        self.live.append((start, nbytes))
        self.pos = (start + nbytes + GUARD + 1023) // 1024 * 1024
        return self.raw[start:start + nbytes]

    def check(self, what: str):
        torch.cuda.synchronize()
        mask = torch.ones(self.raw.numel(), dtype=torch.bool, device="cuda")
        for start, n in self.live:
            mask[start:start + n] = False
        bad = torch.nonzero(mask & (self.raw != PATTERN)).flatten()
        assert bad.numel() == 0, (what, "guard bytes overwritten at arena offsets", bad[:8].tolist(),
                                  "buffers (offset, size):", self.live)


def _stage1_in(arena, B_, w, smooth=True):
    L = B_.lib()
    B, N_q, H_q, N_kv, H_kv = w.B, w.N_q, w.H_q, w.N_kv, w.H_kv
    q4 = B_.Fp4Tensor(arena.take(L.mpfa_fp4_codes_bytes(B, H_q, N_q)), arena.take(L.mpfa_fp4_sf_bytes(B, H_q, N_q)), B, H_q, N_q)
    k4 = B_.Fp4Tensor(arena.take(L.mpfa_fp4_codes_bytes(B, H_kv, N_kv)), arena.take(L.mpfa_fp4_sf_bytes(B, H_kv, N_kv)), B, H_kv, N_kv)
    v8 = arena.take(L.mpfa_v_fp8_bytes(B, H_kv, N_kv))
    delta = arena.take(L.mpfa_delta_s_bytes(B, H_q, N_kv)).view(torch.bfloat16).view(B, H_q, -1)
    stats = B_.Stats(arena.take(B * H_q * 512).view(torch.float32).view(B, H_q, 128),
                     arena.take(B * H_kv * 512).view(torch.float32).view(B, H_kv, 128),
                     arena.take(B * 4).view(torch.float32), arena.take(B * 4).view(torch.float32))
    ws = arena.take(L.mpfa_quantize_workspace_bytes(B, H_q, H_kv))
    s1 = B_.Stage1(q4, k4, v8, delta if smooth else None, stats, 1.0)
    return s1, ws


@pytest.mark.parametrize("arrangement", [0, 1])
def test_stage1_and_prefill_stay_inside_their_buffers(arrangement):
    from paper_2609_33135_b200 import binding as B_
    w = wl.prefill_workload("canary", 91, 2, 333, 4, 2, True, N_q=301, q_bias=True)   # ragged in both lengths
    q, k, v = w.q.cuda(), w.k.cuda(), w.v.cuda()
    ref = B_.stage1(q, k, v)
    B_.mpfa_set_prefill_arrangement(0)
    try:
        ref_out, ref32, st0 = B_.prefill(ref, True, w.softmax_scale, want_f32=True)
    finally:
        B_.mpfa_set_prefill_arrangement(SUITE_ARRANGEMENT)
    arena = Arena(64 << 20)
    s1, ws = _stage1_in(arena, B_, w)
    out = arena.take(w.B * w.N_q * w.H_q * 128 * 2).view(torch.bfloat16).view(w.B, w.N_q, w.H_q, 128)
    o32 = arena.take(w.B * w.N_q * w.H_q * 128 * 4).view(torch.float32).view(w.B, w.N_q, w.H_q, 128)
    status = arena.take(4).view(torch.int32)
    status.zero_()
    arena.check("carving")
    B_.stage1(q, k, v, workspace=ws, out=s1)
    arena.check("stage 1")
    assert torch.equal(s1.q.codes, ref.q.codes) and torch.equal(s1.k.sf, ref.k.sf) and torch.equal(s1.v_fp8, ref.v_fp8)
    assert torch.equal(s1.delta.view(torch.uint16), ref.delta.view(torch.uint16))
    B_.mpfa_set_prefill_arrangement(arrangement)
    try:
        for variant in (0, B_.MPFA_VARIANT_COMP_ELEMENTWISE):
            B_.mpfa_prefill_variant(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, 1.0, True, w.softmax_scale, variant, out, o32, status)
            arena.check(f"prefill variant {variant}, arrangement {arrangement}")
            assert int(status.item()) == 0
        B_.mpfa_prefill(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, 1.0, True, w.softmax_scale, out, o32, status)
        arena.check("prefill")
    finally:
        B_.mpfa_set_prefill_arrangement(SUITE_ARRANGEMENT)
    if arrangement == 0:
        assert torch.equal(out.view(torch.uint16), ref_out.view(torch.uint16)) and torch.equal(o32, ref32)
    # the precision variants' operands and outputs
    L = B_.lib()
    vt = arena.take(2 * L.mpfa_v_fp8_bytes(w.B, w.H_kv, w.N_kv)).view(torch.bfloat16).view(w.B, w.H_kv, -1, 128)
    B_._check(L.mpfa_pack_v_bf16(B_._ptr(v), w.B, w.N_kv, w.H_kv, B_._ptr(vt), B_._stream()), "mpfa_pack_v_bf16")
    v4 = arena.take(L.mpfa_v_fp4_bytes(w.B, w.H_kv, w.N_kv))
    g = float(v.abs().max().float().item()) / (6.0 * 448.0)
    B_._check(L.mpfa_quantize_v_fp4(B_._ptr(v), w.B, w.N_kv, w.H_kv, g, B_._ptr(v4), B_._stream()), "mpfa_quantize_v_fp4")
    arena.check("V operands of the precision variants")
    B_.mpfa_prefill_variant(s1.q, s1.k, vt, s1.delta, s1.stats, 1.0, True, w.softmax_scale, B_.MPFA_VARIANT_PV_BF16, out, o32, status)
    B_.mpfa_prefill_variant(s1.q, s1.k, v4, s1.delta, s1.stats, g, True, w.softmax_scale, B_.MPFA_VARIANT_PV_FP4, out, o32, status)
    arena.check("precision variants")
    assert int(status.item()) == 0


def test_cache_writes_paged_prefill_and_decode_stay_inside_their_buffers():
    from paper_2609_33135_b200 import binding as B_
    L = B_.lib()
    H_q, H_kv = 8, 2
    lens = [200, 65, 1]                       # ragged pages, a one-token context
    Bn = len(lens)
    max_pages = 5
    num_pages = 9
    g = torch.Generator().manual_seed(92)
    arena = Arena(32 << 20)
    kv = B_.PagedKV(arena.take(num_pages * H_kv * 4096).view(num_pages, H_kv, 4096),
                    arena.take(num_pages * H_kv * 512).view(num_pages, H_kv, 512),
                    arena.take(num_pages * H_kv * 8192).view(num_pages, H_kv, 8192),
                    arena.take(num_pages * H_q * 128).view(torch.bfloat16).view(num_pages, H_q, 64), num_pages, H_q, H_kv)
    stats = B_.Stats(arena.take(Bn * H_q * 512).view(torch.float32).view(Bn, H_q, 128),
                     arena.take(Bn * H_kv * 512).view(torch.float32).view(Bn, H_kv, 128),
                     arena.take(Bn * 4).view(torch.float32), arena.take(Bn * 4).view(torch.float32))
    ws = arena.take(L.mpfa_quantize_workspace_bytes(Bn, H_q, H_kv))
    dws = arena.take(L.mpfa_decode_workspace_bytes(Bn, H_q, H_kv, max_pages))
    out = arena.take(Bn * H_q * 128 * 2).view(torch.bfloat16).view(Bn, H_q, 128)
    o32 = arena.take(Bn * H_q * 128 * 4).view(torch.float32).view(Bn, H_q, 128)
    status = arena.take(4).view(torch.int32)
    status.zero_()
    table = torch.tensor([[3, 7, 1, 8, -1], [0, 5, -1, -1, -1], [2, -1, -1, -1, -1]], dtype=torch.int32, device="cuda")
    seq = torch.tensor(lens, dtype=torch.int32, device="cuda")
    qs = torch.randn(Bn, 64, H_q, 128, generator=g).to(torch.bfloat16).cuda()
    scratch = B_.Fp4Tensor(arena.take(L.mpfa_fp4_codes_bytes(Bn, H_q, 64)), arena.take(L.mpfa_fp4_sf_bytes(Bn, H_q, 64)), Bn, H_q, 64)
    B_.mpfa_quantize_qk(qs, None, B_.MPFA_SMOOTH, stats, scratch, None, None, ws)
    arena.check("query statistics")
    for b, n in enumerate(lens):
        k = (torch.randn(n, H_kv, 128, generator=g) + 0.5).to(torch.bfloat16).cuda()
        v = torch.randn(n, H_kv, 128, generator=g).to(torch.bfloat16).cuda()
        first = max(0, n - 3) if n > 3 else 0
        if first:
            B_.mpfa_quantize_kv_paged(k[:first], v[:first], 0, H_q, B_.MPFA_SMOOTH, stats.request(b), 1.0, kv, table[b], ws)
            # the last tokens arrive as an append at a position inside a page (frozen statistics)
            B_.mpfa_quantize_kv_paged(k[first:], v[first:], first, H_q, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, stats.request(b), 1.0,
                                      kv, table[b], None)
        else:
            B_.mpfa_quantize_kv_paged(k, v, 0, H_q, B_.MPFA_SMOOTH, stats.request(b), 1.0, kv, table[b], ws)
        arena.check(f"cache write of request {b}")
    # one more token per request through the batched append (positions = current lengths where a page exists)
    k1 = torch.randn(Bn, 1, H_kv, 128, generator=g).to(torch.bfloat16).cuda()
    v1 = torch.randn(Bn, 1, H_kv, 128, generator=g).to(torch.bfloat16).cuda()
    pos = torch.tensor([200, 65, 1], dtype=torch.int32, device="cuda")
    B_.mpfa_append_kv_paged(k1, v1, H_q, B_.MPFA_SMOOTH, stats, 1.0, kv, table, pos)
    arena.check("batched append")
    seq = seq + 1
    q_new = torch.randn(Bn, 1, H_q, 128, generator=g).to(torch.bfloat16).cuda()
    q4 = B_.Fp4Tensor(arena.take(L.mpfa_fp4_codes_bytes(Bn, H_q, 1)), arena.take(L.mpfa_fp4_sf_bytes(Bn, H_q, 1)), Bn, H_q, 1)
    B_.mpfa_quantize_qk(q_new, None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, stats, q4, None, None, None)
    B_.mpfa_decode(q4, kv, table, seq, stats, 1.0, 128 ** -0.5, out, o32, dws, status)
    arena.check("decode")
    assert int(status.item()) == 0 and torch.isfinite(o32).all()
    # a chunk of queries per request against the same pages
    qc = torch.randn(Bn, 130, H_q, 128, generator=g).to(torch.bfloat16).cuda()
    qc4 = B_.Fp4Tensor(arena.take(L.mpfa_fp4_codes_bytes(Bn, H_q, 130)), arena.take(L.mpfa_fp4_sf_bytes(Bn, H_q, 130)), Bn, H_q, 130)
    B_.mpfa_quantize_qk(qc, None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, stats, qc4, None, None, None)
    pout = arena.take(Bn * 130 * H_q * 128 * 2).view(torch.bfloat16).view(Bn, 130, H_q, 128)
    q_lens = torch.tensor([130, 60, 2], dtype=torch.int32, device="cuda")
    for arrangement in (0, 1):
        B_.mpfa_set_prefill_arrangement(arrangement)
        try:
            B_.mpfa_prefill_paged(qc4, kv, table, seq, stats, 1.0, 128 ** -0.5, pout, None, status, q_lens=q_lens)
            arena.check(f"paged prefill, arrangement {arrangement}")
        finally:
            B_.mpfa_set_prefill_arrangement(SUITE_ARRANGEMENT)
    assert int(status.item()) == 0

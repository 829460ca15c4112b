"""Seeded synthetic inputs for the QK4PV8 attention path.

This module only draws random tensors and index tables.  It contains none of
the method's arithmetic (no centering, no quantization, no softmax) so that
both the CPU oracle's tests and the CUDA path's tests/bench can share it
without sharing any part of the computation.

Value structure (stands in for real model activations, which the paper
describes as ridges along the channel axis that stay flat along tokens,
Section 4.2): Q, K, V ~ N(0, 1); K additionally gets a per-(kv head, channel)
offset b ~ N(0, variance 2) and a few "outlier" channels multiplied by 8.
Everything is rounded to BF16 and magnitudes below 2**-14 are flushed to zero
(this bounds the number of significant bits of any column sum, so a sum of
up to 2**17 tokens is exact in FP64 in every summation order).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

HEAD_DIM = 128
PAGE_SIZE = 64

# sub-stream ids under a config seed
_SUB = dict(q=0, k=1, v=2, bias=3, outlier=4, seq_lens=5, pages=6, rows=7, decode_q=8, qbias=9)


def _gen(seed: int, sub: str) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 16 + _SUB[sub])
    return g


def _finish(x: torch.Tensor) -> torch.Tensor:
    """Round to BF16 and flush |x| < 2**-14 to zero."""
    x = x.to(torch.bfloat16)
    tiny = x.abs().to(torch.float32) < 2.0 ** -14
    return torch.where(tiny, torch.zeros_like(x), x).contiguous()


def _randn_chunked(shape, g: torch.Generator) -> torch.Tensor:
    """randn in FP32, drawn in one call per leading index to bound peak memory."""
    out = torch.empty(shape, dtype=torch.float32)
    flat = out.view(shape[0], -1)
    for i in range(shape[0]):
        flat[i].normal_(generator=g)
    return out


@dataclasses.dataclass
class PrefillWorkload:
    name: str
    B: int
    N_q: int
    N_kv: int
    H_q: int
    H_kv: int
    causal: bool
    softmax_scale: float
    q: torch.Tensor  # [B, N_q, H_q, 128] bf16 (CPU)
    k: torch.Tensor  # [B, N_kv, H_kv, 128] bf16
    v: torch.Tensor  # [B, N_kv, H_kv, 128] bf16

    @property
    def flops(self) -> float:
        """Attention FLOPs, FlashAttention convention: 4*N_q*N_kv*d*H_q, halved when causal."""
        f = 4.0 * self.B * self.N_q * self.N_kv * HEAD_DIM * self.H_q
        return f / 2 if self.causal else f


def k_structure(seed: int, H_kv: int, n_outlier: int):
    """Per-(kv head, channel) additive offset and multiplicative outlier factor for K."""
    bias = torch.empty(H_kv, HEAD_DIM, dtype=torch.float32).normal_(
        mean=0.0, std=math.sqrt(2.0), generator=_gen(seed, "bias"))
    perm = torch.randperm(H_kv * HEAD_DIM, generator=_gen(seed, "outlier"))[:n_outlier]
    factor = torch.ones(H_kv * HEAD_DIM, dtype=torch.float32)
    factor[perm] = 8.0
    return bias, factor.view(H_kv, HEAD_DIM)


def make_qkv(seed: int, B: int, N_q: int, N_kv: int, H_q: int, H_kv: int,
             n_outlier: Optional[int] = None, q_bias: bool = False, device: str = "cpu"):
    """Draw Q [B,N_q,H_q,128], K, V [B,N_kv,H_kv,128] (BF16).  On "cpu" the draw uses the CPU generator; on a CUDA
    device it uses that device's generator with the same seeds (a different but equally reproducible stream),
    which keeps the long benchmark shapes off the host."""
    if n_outlier is None:
        n_outlier = max(1, round(0.01 * H_kv * HEAD_DIM))
    if device != "cpu":
        def draw(sub, n, h):
            g = torch.Generator(device=device)
            g.manual_seed(seed * 16 + _SUB[sub])
            return torch.randn(B, n, h, HEAD_DIM, generator=g, device=device)
        q = draw("q", N_q, H_q)
        if q_bias:
            q = q + torch.empty(H_q, HEAD_DIM, dtype=torch.float32).normal_(
                mean=0.0, std=math.sqrt(2.0), generator=_gen(seed, "qbias")).to(device)
        bias, factor = k_structure(seed, H_kv, n_outlier)
        k = draw("k", N_kv, H_kv) * factor.to(device) + bias.to(device)
        v = draw("v", N_kv, H_kv)
        return _finish(q), _finish(k), _finish(v)
    q = _randn_chunked((B * N_q, H_q, HEAD_DIM), _gen(seed, "q")).view(B, N_q, H_q, HEAD_DIM)
    if q_bias:
        qb = torch.empty(H_q, HEAD_DIM, dtype=torch.float32).normal_(
            mean=0.0, std=math.sqrt(2.0), generator=_gen(seed, "qbias"))
        q = q + qb
    k = _randn_chunked((B * N_kv, H_kv, HEAD_DIM), _gen(seed, "k")).view(B, N_kv, H_kv, HEAD_DIM)
    bias, factor = k_structure(seed, H_kv, n_outlier)
    k = k * factor + bias
    v = _randn_chunked((B * N_kv, H_kv, HEAD_DIM), _gen(seed, "v")).view(B, N_kv, H_kv, HEAD_DIM)
    return _finish(q), _finish(k), _finish(v)


def prefill_workload(name: str, seed: int, B: int, N: int, H_q: int, H_kv: int, causal: bool,
                     n_outlier: Optional[int] = None, q_bias: bool = False,
                     N_q: Optional[int] = None, device: str = "cpu") -> PrefillWorkload:
    N_q = N if N_q is None else N_q
    q, k, v = make_qkv(seed, B, N_q, N, H_q, H_kv, n_outlier, q_bias, device)
    return PrefillWorkload(name, B, N_q, N, H_q, H_kv, causal, 1.0 / math.sqrt(HEAD_DIM), q, k, v)


# The benchmark configurations (shapes from the paper's kernel evaluation, Section 7.2).
def config1_tiny() -> PrefillWorkload:
    return prefill_workload("cfg1_tiny_noncausal_256", 1001, 1, 256, 1, 1, False, n_outlier=4)


def config1b_tiny_qbias() -> PrefillWorkload:
    """Config 1 with a per-channel offset on Q as well, so the query mean (and the
    compensation vector built from it) is far from zero."""
    return prefill_workload("cfg1b_tiny_qbias_256", 1011, 1, 256, 1, 1, False, n_outlier=4, q_bias=True)


def config2_llama(N: int = 16384, seed: int = 1002) -> PrefillWorkload:
    """`seed` selects the batch element (data-parallel ranks take different elements of the same shape)."""
    return prefill_workload(f"cfg2_llama8b_causal_{N}", seed, 1, N, 32, 8, True)


def config3_qwen(N: int = 32768) -> PrefillWorkload:
    return prefill_workload(f"cfg3_qwen14b_causal_{N}", 1003, 1, N, 40, 8, True)


def config4_long(N: int = 131072) -> PrefillWorkload:
    return prefill_workload(f"cfg4_long_causal_{N}", 1004, 1, N, 32, 8, True)


def sample_rows(seed: int, B: int, H_q: int, N_q: int, n_rows: int) -> torch.Tensor:
    """Stratified (batch, q head, query row) sample, int32 [n, 3].

    Always contains rows 0, 127, 128 and N_q-1 (tile edges) of head 0, one row per
    512-row band, and the rest uniformly at random."""
    g = _gen(seed, "rows")
    rows = []
    for r in (0, 127, 128, N_q - 1):
        if 0 <= r < N_q:
            rows.append((0, 0, r))
    band = 512
    for start in range(0, N_q, band):
        r = start + int(torch.randint(0, min(band, N_q - start), (1,), generator=g))
        h = int(torch.randint(0, H_q, (1,), generator=g))
        b = int(torch.randint(0, B, (1,), generator=g))
        rows.append((b, h, r))
    while len(rows) < n_rows:
        rows.append((int(torch.randint(0, B, (1,), generator=g)),
                     int(torch.randint(0, H_q, (1,), generator=g)),
                     int(torch.randint(0, N_q, (1,), generator=g))))
    rows = sorted(set(rows))[:n_rows]
    return torch.tensor(rows, dtype=torch.int32)


@dataclasses.dataclass
class DecodeWorkload:
    name: str
    B: int
    H_q: int
    H_kv: int
    softmax_scale: float
    seq_lens: torch.Tensor      # [B] int32, valid KV tokens per request
    page_table: torch.Tensor    # [B, max_pages] int32 physical page ids (-1 = unused)
    num_pages: int              # size of the physical page pool
    q_sample: torch.Tensor      # [B, N_s, H_q, 128] bf16: tokens the frozen Q statistics come from
    q_new: torch.Tensor         # [B, 1, H_q, 128] bf16: the decode-step query token
    seed: int
    n_outlier: int

    def kv_for_request(self, b: int, device: str = "cpu"):
        """K, V [1, L_b, H_kv, 128] (BF16) of request b, drawn on demand.  On "cpu" the draw
        uses the CPU generator; on a CUDA device it uses that device's generator with the same
        seed (a different but equally reproducible stream), which keeps the 128K-token
        benchmark cache off the host."""
        L = int(self.seq_lens[b])
        s = self.seed * 64 + b
        bias, factor = k_structure(self.seed, self.H_kv, self.n_outlier)
        if device == "cpu":
            k = _randn_chunked((L, self.H_kv, HEAD_DIM), _gen(s, "k")).view(1, L, self.H_kv, HEAD_DIM)
            v = _randn_chunked((L, self.H_kv, HEAD_DIM), _gen(s, "v")).view(1, L, self.H_kv, HEAD_DIM)
        else:
            g = torch.Generator(device=device)
            g.manual_seed(s * 16 + _SUB["k"])
            k = torch.randn(1, L, self.H_kv, HEAD_DIM, generator=g, device=device)
            g.manual_seed(s * 16 + _SUB["v"])
            v = torch.randn(1, L, self.H_kv, HEAD_DIM, generator=g, device=device)
            bias, factor = bias.to(device), factor.to(device)
        k = k * factor + bias
        return _finish(k), _finish(v)

    @property
    def total_tokens(self) -> int:
        return int(self.seq_lens.sum())


def decode_workload(name: str, seed: int, B: int, H_q: int, H_kv: int, len_lo: int, len_hi: int,
                    n_stat_tokens: int = 1024, shuffle_pages: bool = True,
                    extra_pages: int = 3, seq_lens=None) -> DecodeWorkload:
    if seq_lens is None:
        seq_lens = torch.randint(len_lo, len_hi + 1, (B,), generator=_gen(seed, "seq_lens"), dtype=torch.int64)
    else:
        seq_lens = torch.as_tensor(seq_lens, dtype=torch.int64)
        assert seq_lens.shape == (B,)
    pages_per_req = (seq_lens + PAGE_SIZE - 1) // PAGE_SIZE
    total = int(pages_per_req.sum())
    num_pages = total + extra_pages
    if shuffle_pages:
        perm = torch.randperm(num_pages, generator=_gen(seed, "pages"))[:total]
    else:
        perm = torch.arange(total)
    max_pages = int(pages_per_req.max())
    table = torch.full((B, max_pages), -1, dtype=torch.int32)
    off = 0
    for b in range(B):
        n = int(pages_per_req[b])
        table[b, :n] = perm[off:off + n].to(torch.int32)
        off += n
    n_outlier = max(1, round(0.01 * H_kv * HEAD_DIM))
    gq = _gen(seed, "decode_q")
    qs = torch.empty(B, n_stat_tokens + 1, H_q, HEAD_DIM, dtype=torch.float32).normal_(generator=gq)
    qs = _finish(qs)
    return DecodeWorkload(name, B, H_q, H_kv, 1.0 / math.sqrt(HEAD_DIM), seq_lens.to(torch.int32), table,
                          num_pages, qs[:, :n_stat_tokens].contiguous(), qs[:, n_stat_tokens:].contiguous(),
                          seed, n_outlier)


def config5_decode(B: int = 32, len_lo: int = 16384, len_hi: int = 131072) -> DecodeWorkload:
    return decode_workload(f"cfg5_paged_decode_b{B}", 1005, B, 32, 8, len_lo, len_hi)

"""GPU parity: prefill of a chunk of queries against the paged low-bit cache (Section 6: K/V live only in
the quantized pages; a later chunk of a prompt attends to them there) against the oracle's prefill with
N_q < N_kv under the bottom-right aligned causal mask and frozen statistics.  Same tolerance as the
contiguous prefill."""
import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl
from test_gpu_prefill import compare

pytestmark = pytest.mark.gpu


def build_and_run(seed, H_q, H_kv, L, N_q, smooth=True, shuffle=True, q_off=100):
    """Cache = prefix (statistics measured there) + the chunk's own K/V appended with frozen statistics;
    queries = a slice of the request's query sample, quantized with the frozen query statistics."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    B = len(L)
    L0 = [l - N_q for l in L]
    assert min(L0) >= 1
    w_full = wl.decode_workload("pp", seed, B, H_q, H_kv, 1, max(L), seq_lens=L, shuffle_pages=shuffle)
    w0 = wl.decode_workload("pp", seed, B, H_q, H_kv, 1, max(L), seq_lens=L0, shuffle_pages=shuffle)
    w0.page_table, w0.num_pages = w_full.page_table, w_full.num_pages
    kv_full = [w_full.kv_for_request(b) for b in range(B)]
    w0.kv_for_request = lambda b, device="cpu": (kv_full[b][0][:, :L0[b]].contiguous(), kv_full[b][1][:, :L0[b]].contiguous())
    st = decode_cache.build_cache(w0, smooth=smooth)
    flags = (B_.MPFA_SMOOTH if smooth else 0) | B_.MPFA_STATS_FROZEN
    for b in range(B):
        k, v = kv_full[b][0][0].cuda(), kv_full[b][1][0].cuda()
        B_.mpfa_quantize_kv_paged(k[L0[b]:].contiguous(), v[L0[b]:].contiguous(), L0[b], H_q, flags,
                                  st.stats.request(b), 1.0, st.kv, st.page_table[b], None)
    q_chunk = w_full.q_sample[:, q_off:q_off + N_q].contiguous()
    q4 = B_.Fp4Tensor.empty(B, H_q, N_q, "cuda")
    B_.mpfa_quantize_qk(q_chunk.cuda(), None, flags, st.stats, q4, None, None, None)
    out = torch.empty(B, N_q, H_q, 128, dtype=torch.bfloat16, device="cuda")
    o32 = torch.empty(B, N_q, H_q, 128, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    seq = torch.tensor(L, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_paged(q4, st.kv, st.page_table, seq, st.stats, 1.0, w_full.softmax_scale, out, o32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    refs = []
    for b in range(B):
        kb, vb = kv_full[b]
        z0 = orc.stage1(orc.bf16_bits(w_full.q_sample[b:b + 1].contiguous()), orc.bf16_bits(kb[:, :L0[b]].contiguous()),
                        orc.bf16_bits(vb[:, :L0[b]].contiguous()), smooth=smooth)
        z = orc.stage1(orc.bf16_bits(q_chunk[b:b + 1].contiguous()), orc.bf16_bits(kb), orc.bf16_bits(vb), smooth=smooth,
                       frozen=z0)
        refs.append(z)
    return w_full, out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy(), refs


@pytest.mark.parametrize("name,H_q,H_kv,L,N_q", [
    ("one_tile", 4, 2, [200], 100),
    ("ragged_gqa4", 8, 2, [391, 200, 700], 150),           # odd and even page counts, ragged last block, two q tiles
    ("gqa8_aligned", 8, 1, [1024, 512], 256),              # block-aligned contexts, every swizzle of Delta_S
    ("mha_long_prefix", 2, 2, [4500, 2300], 130),          # many KV blocks per item: several page look-up groups
    ("gqa5", 10, 2, [333, 650], 129),
])
def test_paged_prefill_matches_oracle(name, H_q, H_kv, L, N_q):
    w, o16, o32, refs = build_and_run(300 + len(name), H_q, H_kv, L, N_q)
    for b, z in enumerate(refs):
        rows = orc.all_rows(1, H_q, N_q)
        if len(rows) > 1200:   # long prefixes: a stratified sample of rows, always with the tile edges
            keep = np.unique(np.concatenate([np.arange(0, len(rows), max(1, len(rows) // 600)),
                                             [0, N_q - 1, min(127, N_q - 1), min(128, N_q - 1), len(rows) - 1]]))
            rows = rows[keep]
        ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
        compare(o16[b:b + 1], o32[b:b + 1], rows, ref32, f"{name} request {b}")


def test_paged_prefill_without_compensation():
    """Cache without a Delta_S pool (the direct variant: no smoothing, no compensation MMA)."""
    w, o16, o32, refs = build_and_run(321, 4, 2, [300, 170], 90, smooth=False)
    for b, z in enumerate(refs):
        rows = orc.all_rows(1, 4, 90)
        ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
        compare(o16[b:b + 1], o32[b:b + 1], rows, ref32, f"direct request {b}")


def test_paged_prefill_equals_contiguous_prefill_bitwise():
    """The paged source changes where the operand tiles come from, not the arithmetic: with the whole prompt as
    the chunk (no frozen prefix needed: statistics of the full tensors), the output must equal the contiguous
    prefill's bit for bit."""
    from paper_2609_33135_b200 import binding as B_
    w = wl.prefill_workload("ppeq", 71, 1, 777, 8, 2, True, q_bias=True)
    s1 = B_.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda())
    out_c, o32_c, status = B_.prefill(s1, True, w.softmax_scale, want_f32=True)
    n_pages = (777 + 63) // 64
    kv = B_.PagedKV.empty(n_pages + 2, 8, 2, with_delta=True, device="cuda")
    table = torch.arange(n_pages - 1, -1, -1, dtype=torch.int32, device="cuda").view(1, -1).contiguous()   # reversed pool order
    B_.mpfa_quantize_kv_paged(w.k[0].cuda(), w.v[0].cuda(), 0, 8, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, s1.stats.request(0), 1.0,
                              kv, table[0], None)
    out_p = torch.empty_like(out_c)
    o32_p = torch.empty_like(o32_c)
    st2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_paged(s1.q, kv, table, torch.tensor([777], dtype=torch.int32, device="cuda"), s1.stats, 1.0,
                          w.softmax_scale, out_p, o32_p, st2)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and int(st2.item()) == 0
    assert torch.equal(o32_p.view(torch.int32), o32_c.view(torch.int32))
    assert torch.equal(out_p.view(torch.uint16), out_c.view(torch.uint16))


def test_paged_prefill_bad_page_is_reported_not_followed():
    from paper_2609_33135_b200 import binding as B_
    w, _, _, _ = build_and_run(333, 4, 2, [200], 100)
    # same call again with a page id outside the pool
    from paper_2609_33135_b200 import decode_cache
    st = decode_cache.build_cache(w)
    table = st.page_table.clone()
    table[0, 1] = w.num_pages + 5
    q4 = B_.Fp4Tensor.empty(1, 4, 100, "cuda")
    B_.mpfa_quantize_qk(w.q_sample[:, :100].contiguous().cuda(), None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats, q4,
                        None, None, None)
    out = torch.empty(1, 100, 4, 128, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_paged(q4, st.kv, table, st.seq_lens, st.stats, 1.0, w.softmax_scale, out, None, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B_.MPFA_DEV_BAD_PAGE


def test_paged_prefill_more_queries_than_keys():
    """Degenerate case: a chunk longer than the request's whole context (bottom-right aligned mask: the first
    N_q - L rows see no key and must come out as zeros, a whole query tile may have no KV block at all) next to an
    ordinary request in the same launch."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    L, N_q, H_q, H_kv = [50, 300], 200, 4, 2
    w = wl.decode_workload("pp_short", 341, 2, H_q, H_kv, 1, 300, seq_lens=L)
    st = decode_cache.build_cache(w)
    q_chunk = w.q_sample[:, 10:10 + N_q].contiguous()
    q4 = B_.Fp4Tensor.empty(2, H_q, N_q, "cuda")
    B_.mpfa_quantize_qk(q_chunk.cuda(), None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats, q4, None, None, None)
    out = torch.full((2, N_q, H_q, 128), 3.0, dtype=torch.bfloat16, device="cuda")
    o32 = torch.full((2, N_q, H_q, 128), 3.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_paged(q4, st.kv, st.page_table, st.seq_lens, st.stats, 1.0, w.softmax_scale, out, o32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o16n, o32n = out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy()
    assert not o32n[0, :N_q - 50].any() and not o16n[0, :N_q - 50].any()
    for b in range(2):
        k, v = w.kv_for_request(b)
        z0 = orc.stage1(orc.bf16_bits(w.q_sample[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v))
        z = orc.stage1(orc.bf16_bits(q_chunk[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v), frozen=z0)
        rows = orc.all_rows(1, H_q, N_q)
        ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
        compare(o16n[b:b + 1], o32n[b:b + 1], rows, ref32, f"request {b}")


def test_paged_prefill_batch_of_chunks_of_different_lengths():
    """Requests with different numbers of new queries in one launch (q_lens): request b's queries are the first
    q_lens[b] rows of its slab and the last q_lens[b] tokens of its context; rows past that come out as zeros.
    Includes a request with no query at all and one whose count ends inside a query tile."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    H_q, H_kv, N_q = 8, 2, 150
    L, QL = [391, 200, 700, 90], [150, 37, 129, 0]
    B = len(L)
    w = wl.decode_workload("pp_varlen", 351, B, H_q, H_kv, 1, max(L), seq_lens=L)
    st = decode_cache.build_cache(w)   # whole contexts in the cache; statistics frozen from them
    q_all = w.q_sample[:, 200:200 + N_q].contiguous()
    q4 = B_.Fp4Tensor.empty(B, H_q, N_q, "cuda")
    B_.mpfa_quantize_qk(q_all.cuda(), None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats, q4, None, None, None)
    out = torch.full((B, N_q, H_q, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    o32 = torch.full((B, N_q, H_q, 128), 5.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_paged(q4, st.kv, st.page_table, st.seq_lens, st.stats, 1.0, w.softmax_scale, out, o32, status,
                          q_lens=torch.tensor(QL, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o16n, o32n = out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy()
    for b in range(B):
        assert not o32n[b, QL[b]:].any() and not o16n[b, QL[b]:].any(), b
        if QL[b] == 0:
            continue
        k, v = w.kv_for_request(b)
        z0 = orc.stage1(orc.bf16_bits(w.q_sample[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v))
        z = orc.stage1(orc.bf16_bits(q_all[b:b + 1, :QL[b]].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v), frozen=z0)
        rows = orc.all_rows(1, H_q, QL[b])
        ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
        compare(o16n[b:b + 1], o32n[b:b + 1], rows, ref32, f"request {b}")


def test_paged_prefill_length_beyond_the_page_table_is_cut_not_followed():
    """A seq_lens entry larger than the page-table row can address must not make the kernel read past the row: the
    length is treated as 64 * max_pages (here the same as the true length, so the result is unchanged)."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    w = wl.decode_workload("pp_clip", 361, 1, 4, 2, 1, 256, seq_lens=[256])   # exactly 4 pages, table row of 4
    st = decode_cache.build_cache(w)
    q4 = B_.Fp4Tensor.empty(1, 4, 64, "cuda")
    B_.mpfa_quantize_qk(w.q_sample[:, :64].contiguous().cuda(), None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats, q4,
                        None, None, None)
    outs = []
    for L in (256, 100000):
        out = torch.empty(1, 64, 4, 128, dtype=torch.bfloat16, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B_.mpfa_prefill_paged(q4, st.kv, st.page_table, torch.tensor([L], dtype=torch.int32, device="cuda"), st.stats, 1.0,
                              w.softmax_scale, out, None, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs.append(out)
    assert torch.equal(outs[0].view(torch.uint16), outs[1].view(torch.uint16))


def test_paged_prefill_many_query_tiles_past_the_request_length():
    """q_lens far below N_q (128 queries of 8192 slots, 32 heads): 63 of 64 query tiles of every head are empty work
    items that precede the live ones in every CTA's list.  Zeros there, oracle parity on the live rows, status 0."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    H_q, H_kv, N_q, L = 32, 8, 8192, 1000
    w = wl.decode_workload("pp_empty", 371, 1, H_q, H_kv, 1, L, seq_lens=[L], n_stat_tokens=256)
    st = decode_cache.build_cache(w)
    q_live = w.q_sample[:, :128].contiguous()
    q_all = torch.zeros(1, N_q, H_q, 128, dtype=torch.bfloat16)
    q_all[:, :128] = q_live
    q4 = B_.Fp4Tensor.empty(1, H_q, N_q, "cuda")
    B_.mpfa_quantize_qk(q_all.cuda(), None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats, q4, None, None, None)
    out = torch.full((1, N_q, H_q, 128), 5.0, dtype=torch.bfloat16, device="cuda")
    o32 = torch.full((1, N_q, H_q, 128), 5.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_paged(q4, st.kv, st.page_table, st.seq_lens, st.stats, 1.0, w.softmax_scale, out, o32, status,
                          q_lens=torch.tensor([128], dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o16n, o32n = out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy()
    assert not o32n[0, 128:].any() and not o16n[0, 128:].any()
    k, v = w.kv_for_request(0)
    z0 = orc.stage1(orc.bf16_bits(w.q_sample[0:1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v))
    z = orc.stage1(orc.bf16_bits(q_live), orc.bf16_bits(k), orc.bf16_bits(v), frozen=z0)
    rows = orc.all_rows(1, H_q, 128)
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    compare(o16n[:, :128], o32n[:, :128], rows, ref32, "live tile")

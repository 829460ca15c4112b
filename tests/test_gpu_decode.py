"""GPU parity: paged cache write (bit-exact) and split-KV decode (tolerance) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

from layouts import paged_delta_to_logical, paged_k_to_logical, paged_v_to_logical
from test_gpu_prefill import MAX_ABS, MEAN_ABS, bf16_neighbours_ok

pytestmark = pytest.mark.gpu


def oracle_decode(w, smooth=True, v_scale=1.0):
    """Per request: stage 1 with the frozen query statistics, then the partitioned main loop."""
    outs32, outs16, caches = [], [], []
    for b in range(w.B):
        k, v = w.kv_for_request(b)
        qs = w.q_sample[b:b + 1].contiguous()
        z = orc.stage1(orc.bf16_bits(qs), orc.bf16_bits(k), orc.bf16_bits(v), smooth=smooth, v_scale=v_scale)
        zq = orc.stage1(orc.bf16_bits(w.q_new[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v),
                        smooth=smooth, v_scale=v_scale, frozen=z)
        o32, o16 = orc.decode(zq.q_codes[:, :, 0], zq.q_sf[:, :, 0], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq,
                              z.dk, v_scale, w.softmax_scale, np.array([int(w.seq_lens[b])], np.int32))
        outs32.append(o32[0])
        outs16.append(o16[0])
        caches.append(z)
    return np.stack(outs32), np.stack(outs16), caches


def check_cache(state, w, caches, smooth=True):
    kc = state.kv.k_codes.cpu().numpy()
    ks = state.kv.k_sf.cpu().numpy()
    vv = state.kv.v_fp8.cpu().numpy()
    dl = state.kv.delta.view(torch.uint16).cpu().numpy() if smooth else None
    for b in range(w.B):
        z, L = caches[b], int(w.seq_lens[b])
        for i in range((L + 63) // 64):
            page = int(w.page_table[b, i])
            n = min(64, L - 64 * i)
            lk = paged_k_to_logical(kc[page])          # [H_kv, 64, 64]
            lv = paged_v_to_logical(vv[page])          # [H_kv, 64, 128]
            assert np.array_equal(lk[:, :n], z.k_codes[0, :, 64 * i:64 * i + n])
            assert np.array_equal(ks[page].reshape(w.H_kv, 64, 8)[:, :n], z.k_sf[0, :, 64 * i:64 * i + n])
            assert np.array_equal(lv[:, :n], z.v_codes[0, :, 64 * i:64 * i + n])
            assert not lk[:, n:].any() and not lv[:, n:].any()
            if smooth:
                ld = paged_delta_to_logical(dl[page], w.H_q // w.H_kv)
                assert np.array_equal(ld[:, :n], z.delta[0, :, 64 * i:64 * i + n])
                assert not ld[:, n:].any()


def run(w, smooth=True, v_scale=1.0):
    from paper_2609_33135_b200 import decode_cache
    st = decode_cache.build_cache(w, smooth=smooth, v_scale=v_scale)
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    return st


def compare(st, ref32):
    g32 = st.out_f32.cpu().numpy()
    g16 = st.out.view(torch.uint16).cpu().numpy()
    d = np.abs(g32 - ref32)
    assert np.isfinite(g32).all()
    assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (float(d.max()), float(d.mean()))
    assert np.array_equal(g16, torch.from_numpy(g32.copy()).to(torch.bfloat16).view(torch.uint16).numpy())
    assert bf16_neighbours_ok(g16, ref32).all()


@pytest.mark.parametrize("hq,hkv", [(8, 2), (10, 2), (4, 4), (4, 2), (6, 2), (12, 2), (14, 2), (16, 2)])
def test_decode_matches_oracle(hq, hkv):   # every GQA group size 1..8 (the kernel is specialised on it)
    # lengths that hit the edges: one key, one page, one block + 1, one partition + 1, ragged multi-partition
    w = wl.decode_workload("dec_small", 61 + hq, 5, hq, hkv, 1, 2600, seq_lens=[1, 64, 129, 1025, 2600])
    ref32, ref16, caches = oracle_decode(w)
    st = run(w)
    check_cache(st, w, caches)
    compare(st, ref32)


def oracle_decode_one(w, b):
    k, v = w.kv_for_request(b)
    z = orc.stage1(orc.bf16_bits(w.q_sample[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v))
    zq = orc.stage1(orc.bf16_bits(w.q_new[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v), frozen=z)
    o32, _ = orc.decode(zq.q_codes[:, :, 0], zq.q_sf[:, :, 0], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0,
                        w.softmax_scale, np.array([int(w.seq_lens[b])], np.int32))
    return o32[0]


def test_decode_many_short_requests():
    """More requests than the kernel caches lengths for (768), far more work items than CTAs, most of them
    a single partial block: the persistent work walk, the item-boundary hand-offs and the table fallback."""
    B = 800
    w = wl.decode_workload("dec_many", 75, B, 4, 2, 1, 200, n_stat_tokens=64)
    st = run(w)
    got = st.out_f32.cpu().numpy()
    assert np.isfinite(got).all()
    for b in list(range(0, B, 37)) + [767, 768, 769, B - 1]:
        d = np.abs(got[b] - oracle_decode_one(w, b))
        assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (b, float(d.max()), float(d.mean()))


def test_decode_long_request_many_partitions():
    """One request of 20 partitions next to a one-token request: many items per (request, head), merge kernel
    over many partition states."""
    w = wl.decode_workload("dec_long", 76, 2, 8, 2, 1, 20000, seq_lens=[19999, 1])
    st = run(w)
    got = st.out_f32.cpu().numpy()
    for b in range(2):
        d = np.abs(got[b] - oracle_decode_one(w, b))
        assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (b, float(d.max()), float(d.mean()))


def test_decode_direct_variant_and_v_scale():
    w = wl.decode_workload("dec_direct", 71, 3, 8, 2, 300, 3000)
    ref32, _, caches = oracle_decode(w, smooth=False, v_scale=0.5)
    st = run(w, smooth=False, v_scale=0.5)
    check_cache(st, w, caches, smooth=False)
    compare(st, ref32)


def test_decode_independent_of_page_permutation_and_repeatable():
    w1 = wl.decode_workload("dec_perm", 72, 3, 8, 2, 500, 2500, shuffle_pages=True)
    w2 = wl.decode_workload("dec_perm", 72, 3, 8, 2, 500, 2500, shuffle_pages=False)
    assert not torch.equal(w1.page_table, w2.page_table)
    a, b = run(w1), run(w2)
    assert torch.equal(a.out, b.out) and torch.equal(a.out_f32, b.out_f32)
    from paper_2609_33135_b200 import decode_cache
    first = a.out_f32.clone()
    decode_cache.decode_step(a)
    torch.cuda.synchronize()
    assert torch.equal(first, a.out_f32)


def test_decode_bad_page_is_reported_not_followed():
    from paper_2609_33135_b200 import decode_cache
    w = wl.decode_workload("dec_bad", 73, 2, 8, 2, 200, 400)
    st = run(w)
    st.page_table[1, 1] = st.kv.num_pages + 5
    st.status.zero_()
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert int(st.status.item()) & 2
    assert torch.isfinite(st.out_f32).all()


def test_append_into_partly_filled_pages_then_decode():
    """Decode-time appends: a cache built from the first L0 tokens (statistics frozen there) grows token by token
    and in ragged chunks, across page boundaries and into fresh pages; every slab must equal what the oracle
    quantizes for the full sequence with the same frozen statistics (bit-exact), pad slots stay zero, and the
    decode over the grown cache matches the oracle's."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    L0, L1 = [100, 64, 1], [391, 200, 131]
    w_full = wl.decode_workload("dec_append", 77, 3, 8, 2, 1, 400, seq_lens=L1)
    w0 = wl.decode_workload("dec_append", 77, 3, 8, 2, 1, 400, seq_lens=L0)
    # same page pool and table for both: allocate for the final lengths, fill only the first L0 tokens
    w0.page_table, w0.num_pages = w_full.page_table, w_full.num_pages
    kv_full = [w_full.kv_for_request(b) for b in range(3)]
    w0.kv_for_request = lambda b, device="cpu": (kv_full[b][0][:, :L0[b]].contiguous(), kv_full[b][1][:, :L0[b]].contiguous())
    st = decode_cache.build_cache(w0)
    # poison the pages that the appends will start, so that missing zero-fill shows
    for b in range(3):
        for i in range((L0[b] + 63) // 64, (L1[b] + 63) // 64):
            pg = int(w_full.page_table[b, i])
            st.kv.k_codes[pg].fill_(0x7F)
            st.kv.k_sf[pg].fill_(0x7F)
            st.kv.v_fp8[pg].fill_(0x7F)
            st.kv.delta[pg].fill_(float("nan"))
    flags = B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN
    for b in range(3):
        k, v = kv_full[b][0][0].cuda(), kv_full[b][1][0].cuda()
        pos, step = L0[b], 1
        while pos < L1[b]:
            n = min(step, L1[b] - pos)
            B_.mpfa_quantize_kv_paged(k[pos:pos + n].contiguous(), v[pos:pos + n].contiguous(), pos, w_full.H_q, flags,
                                      st.stats.request(b), 1.0, st.kv, st.page_table[b], None)
            pos += n
            step = step % 37 + 5 if pos > L0[b] + 3 else 1   # a few single tokens, then ragged chunks
    torch.cuda.synchronize()
    # oracle: statistics from the first L0 tokens, then everything quantized with them
    caches, refs = [], []
    for b in range(3):
        kb, vb = kv_full[b]
        z0 = orc.stage1(orc.bf16_bits(w_full.q_sample[b:b + 1].contiguous()), orc.bf16_bits(kb[:, :L0[b]].contiguous()),
                        orc.bf16_bits(vb[:, :L0[b]].contiguous()))
        z = orc.stage1(orc.bf16_bits(w_full.q_sample[b:b + 1].contiguous()), orc.bf16_bits(kb), orc.bf16_bits(vb), frozen=z0)
        zq = orc.stage1(orc.bf16_bits(w_full.q_new[b:b + 1].contiguous()), orc.bf16_bits(kb), orc.bf16_bits(vb), frozen=z0)
        o32, _ = orc.decode(zq.q_codes[:, :, 0], zq.q_sf[:, :, 0], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0,
                            w_full.softmax_scale, np.array([L1[b]], np.int32))
        caches.append(z)
        refs.append(o32[0])
    st.w = w_full
    check_cache(st, w_full, caches)
    st.seq_lens.copy_(w_full.seq_lens.to(st.seq_lens.device))
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    compare(st, np.stack(refs))


def test_decode_replays_from_a_cuda_graph():
    """Section 5.3: the decode launch sequence (counter reset, split kernel, merge kernel) has a fixed shape, so
    it can be captured once and replayed while sequence lengths, queries and cache contents change in place."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    w = wl.decode_workload("dec_graph", 91, 4, 8, 2, 300, 3000)
    st = decode_cache.build_cache(w)
    decode_cache.decode_step(st)          # eager run first: loads the kernels outside the capture
    torch.cuda.synchronize()
    eager_full = st.out.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        decode_cache.decode_step(st)
    st.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    assert torch.equal(st.out.view(torch.uint16), eager_full.view(torch.uint16))
    # shorter contexts and another query, written in place; the captured launches are reused unchanged
    shorter = (w.seq_lens // 3 + 1).to(torch.int32)
    st.seq_lens.copy_(shorter.to(st.seq_lens.device))
    q2 = w.q_sample[:, 5:6].contiguous().cuda()
    B_.mpfa_quantize_qk(q2, None, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats, st.q4, None, None, None)
    graph.replay()
    torch.cuda.synchronize()
    from_graph = st.out.clone()
    st.out.zero_()
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    assert torch.equal(from_graph.view(torch.uint16), st.out.view(torch.uint16))
    assert not torch.equal(from_graph.view(torch.uint16), eager_full.view(torch.uint16))


def test_decode_with_empty_contexts_in_the_batch():
    """Degenerate case: requests whose context length is 0 (nothing to attend to) next to ordinary ones.  They
    contribute no work item, their output is defined as zero, and the neighbours are unaffected."""
    from paper_2609_33135_b200 import decode_cache
    w = wl.decode_workload("dec_empty", 92, 5, 8, 2, 1, 1500, seq_lens=[5, 1300, 9, 1, 64])
    st = decode_cache.build_cache(w)
    st.seq_lens.copy_(torch.tensor([0, 1300, 0, 1, 0], dtype=torch.int32).to(st.seq_lens.device))
    st.out.fill_(7.0)
    st.out_f32.fill_(7.0)
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    got = st.out_f32.cpu().numpy()
    for b in (0, 2, 4):
        assert not got[b].any() and not st.out[b].float().cpu().numpy().any()
    for b in (1, 3):
        d = np.abs(got[b] - oracle_decode_one(w, b))
        assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (b, float(d.max()), float(d.mean()))


def test_decode_loop_append_one_token_then_attend():
    """The decode configuration sustained over several steps (Section 6): every step appends one new token per
    request to its pages with the frozen statistics, raises the request's length and decodes; each step's output is
    compared with the oracle's decode over the same prefix."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    L0, steps = [127, 64, 1000], 5
    L1 = [l + steps for l in L0]
    w_full = wl.decode_workload("dec_loop", 93, 3, 8, 2, 1, max(L1), seq_lens=L1)
    w0 = wl.decode_workload("dec_loop", 93, 3, 8, 2, 1, max(L1), seq_lens=L0)
    w0.page_table, w0.num_pages = w_full.page_table, w_full.num_pages
    kv_full = [w_full.kv_for_request(b) for b in range(3)]
    w0.kv_for_request = lambda b, device="cpu": (kv_full[b][0][:, :L0[b]].contiguous(), kv_full[b][1][:, :L0[b]].contiguous())
    st = decode_cache.build_cache(w0)
    st.w = w_full
    flags = B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN
    z0 = [orc.stage1(orc.bf16_bits(w_full.q_sample[b:b + 1].contiguous()), orc.bf16_bits(kv_full[b][0][:, :L0[b]].contiguous()),
                     orc.bf16_bits(kv_full[b][1][:, :L0[b]].contiguous())) for b in range(3)]
    kd = [(kv_full[b][0][0].cuda(), kv_full[b][1][0].cuda()) for b in range(3)]
    for s in range(steps):
        if s % 2 == 0:   # the whole batch in one launch
            k_new = torch.stack([kd[b][0][L0[b] + s:L0[b] + s + 1] for b in range(3)]).contiguous()
            v_new = torch.stack([kd[b][1][L0[b] + s:L0[b] + s + 1] for b in range(3)]).contiguous()
            pos = torch.tensor([l + s for l in L0], dtype=torch.int32, device="cuda")
            B_.mpfa_append_kv_paged(k_new, v_new, w_full.H_q, B_.MPFA_SMOOTH, st.stats, 1.0, st.kv, st.page_table, pos)
        else:            # request by request
            for b in range(3):
                pos = L0[b] + s
                B_.mpfa_quantize_kv_paged(kd[b][0][pos:pos + 1].contiguous(), kd[b][1][pos:pos + 1].contiguous(), pos,
                                          w_full.H_q, flags, st.stats.request(b), 1.0, st.kv, st.page_table[b], None)
        lens = torch.tensor([l + s + 1 for l in L0], dtype=torch.int32)
        st.seq_lens.copy_(lens.to(st.seq_lens.device))
        q_step = w_full.q_sample[:, 10 + s:11 + s].contiguous()
        B_.mpfa_quantize_qk(q_step.cuda(), None, flags, st.stats, st.q4, None, None, None)
        decode_cache.decode_step(st)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        got = st.out_f32.cpu().numpy()
        for b in range(3):
            n = int(lens[b])
            kb, vb = kv_full[b][0][:, :n].contiguous(), kv_full[b][1][:, :n].contiguous()
            z = orc.stage1(orc.bf16_bits(q_step[b:b + 1].contiguous()), orc.bf16_bits(kb), orc.bf16_bits(vb), frozen=z0[b])
            ref, _ = orc.decode(z.q_codes[:, :, 0], z.q_sf[:, :, 0], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0,
                                w_full.softmax_scale, np.array([n], np.int32))
            d = np.abs(got[b] - ref[0])
            assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (s, b, float(d.max()), float(d.mean()))


def test_batched_append_writes_the_same_bytes_as_per_request_appends():
    """mpfa_append_kv_paged against mpfa_quantize_kv_paged with one token: every pool byte equal, over positions that
    start a page (the rest of the page is zeroed), end a page, and with one request skipped (negative position)."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    L0 = [64, 63, 200, 5]          # request 0 starts a new page, request 1 fills the last slot of its page
    w_full = wl.decode_workload("dec_batch_append", 94, 4, 8, 2, 1, 300, seq_lens=[l + 3 for l in L0])
    kv_full = [w_full.kv_for_request(b) for b in range(4)]
    states = []
    for mode in ("batched", "single"):
        w0 = wl.decode_workload("dec_batch_append", 94, 4, 8, 2, 1, 300, seq_lens=L0)
        w0.page_table, w0.num_pages = w_full.page_table, w_full.num_pages
        w0.kv_for_request = lambda b, device="cpu": (kv_full[b][0][:, :L0[b]].contiguous(), kv_full[b][1][:, :L0[b]].contiguous())
        st = decode_cache.build_cache(w0)
        for t in (st.kv.k_codes, st.kv.k_sf, st.kv.v_fp8):   # stale bytes in the pages the appends will start
            t[int(w_full.page_table[0, 1])].fill_(0x7F)
        st.kv.delta[int(w_full.page_table[0, 1])].fill_(float("nan"))
        for s in range(3):
            active = [b for b in range(4) if not (b == 3 and s == 1)]   # request 3 sits out step 1
            if mode == "batched":
                k_new = torch.stack([kv_full[b][0][0, L0[b] + s:L0[b] + s + 1] for b in range(4)]).contiguous().cuda()
                v_new = torch.stack([kv_full[b][1][0, L0[b] + s:L0[b] + s + 1] for b in range(4)]).contiguous().cuda()
                pos = torch.tensor([L0[b] + s if b in active else -1 for b in range(4)], dtype=torch.int32, device="cuda")
                B_.mpfa_append_kv_paged(k_new, v_new, w_full.H_q, B_.MPFA_SMOOTH, st.stats, 1.0, st.kv, st.page_table, pos)
            else:
                for b in active:
                    p = L0[b] + s
                    B_.mpfa_quantize_kv_paged(kv_full[b][0][0, p:p + 1].contiguous().cuda(), kv_full[b][1][0, p:p + 1].contiguous().cuda(),
                                              p, w_full.H_q, B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN, st.stats.request(b), 1.0,
                                              st.kv, st.page_table[b], None)
        torch.cuda.synchronize()
        states.append(st)
    a, b = states
    used = sorted({int(p) for r in range(4) for p in w_full.page_table[r] if int(p) >= 0})
    for name in ("k_codes", "k_sf", "v_fp8"):
        assert torch.equal(getattr(a.kv, name)[used], getattr(b.kv, name)[used]), name
    assert torch.equal(a.kv.delta[used].view(torch.int16), b.kv.delta[used].view(torch.int16))
    pg = int(w_full.page_table[0, 1])
    assert not a.kv.k_codes[pg].view(-1, 4096)[:, :].reshape(2, 8, 512)[:, 1:].any()   # slots 8.. of the started page are zero


def test_serving_step_captured_once_and_replayed():
    """The whole decode-time step - write the batch's new K/V token into the pages, quantize the new query with the
    frozen statistics, attend - captured in one CUDA graph and replayed: positions, inputs and lengths change in
    place between replays; every replay is compared with the oracle."""
    from paper_2609_33135_b200 import binding as B_, decode_cache
    L0, steps = [190, 63, 2047], 4
    L1 = [l + steps for l in L0]
    w_full = wl.decode_workload("dec_graph_step", 95, 3, 8, 2, 1, max(L1), seq_lens=L1)
    w0 = wl.decode_workload("dec_graph_step", 95, 3, 8, 2, 1, max(L1), seq_lens=L0)
    w0.page_table, w0.num_pages = w_full.page_table, w_full.num_pages
    kv_full = [w_full.kv_for_request(b) for b in range(3)]
    w0.kv_for_request = lambda b, device="cpu": (kv_full[b][0][:, :L0[b]].contiguous(), kv_full[b][1][:, :L0[b]].contiguous())
    st = decode_cache.build_cache(w0)
    flags = B_.MPFA_SMOOTH | B_.MPFA_STATS_FROZEN
    z0 = [orc.stage1(orc.bf16_bits(w_full.q_sample[b:b + 1].contiguous()), orc.bf16_bits(kv_full[b][0][:, :L0[b]].contiguous()),
                     orc.bf16_bits(kv_full[b][1][:, :L0[b]].contiguous())) for b in range(3)]
    k_new = torch.empty(3, 1, 2, 128, dtype=torch.bfloat16, device="cuda")
    v_new = torch.empty_like(k_new)
    q_new = torch.empty(3, 1, 8, 128, dtype=torch.bfloat16, device="cuda")
    pos = torch.tensor(L0, dtype=torch.int32, device="cuda")

    def step():
        B_.mpfa_append_kv_paged(k_new, v_new, w_full.H_q, B_.MPFA_SMOOTH, st.stats, 1.0, st.kv, st.page_table, pos)
        torch.add(pos, 1, out=st.seq_lens)
        B_.mpfa_quantize_qk(q_new, None, flags, st.stats, st.q4, None, None, None)
        decode_cache.decode_step(st)

    def load_inputs(s):
        k_new.copy_(torch.stack([kv_full[b][0][0, L0[b] + s:L0[b] + s + 1] for b in range(3)]))
        v_new.copy_(torch.stack([kv_full[b][1][0, L0[b] + s:L0[b] + s + 1] for b in range(3)]))
        q_new.copy_(w_full.q_sample[:, 20 + s:21 + s])
        pos.copy_(torch.tensor([l + s for l in L0], dtype=torch.int32))

    load_inputs(0)
    step()                      # eager once: loads the kernels outside the capture (idempotent: same token, same slot)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for s in range(steps):
        load_inputs(s)
        graph.replay()
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        got = st.out_f32.cpu().numpy()
        for b in range(3):
            n = L0[b] + s + 1
            kb, vb = kv_full[b][0][:, :n].contiguous(), kv_full[b][1][:, :n].contiguous()
            z = orc.stage1(orc.bf16_bits(w_full.q_sample[b:b + 1, 20 + s:21 + s].contiguous()), orc.bf16_bits(kb), orc.bf16_bits(vb),
                           frozen=z0[b])
            ref, _ = orc.decode(z.q_codes[:, :, 0], z.q_sf[:, :, 0], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0,
                                w_full.softmax_scale, np.array([n], np.int32))
            d = np.abs(got[b] - ref[0])
            assert d.max() <= MAX_ABS and d.mean() <= MEAN_ABS, (s, b, float(d.max()), float(d.mean()))

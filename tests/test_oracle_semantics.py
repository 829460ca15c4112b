"""Pins for three semantics of the oracle's attention loop that a tolerance test cannot see:
the reverse traversal of the KV blocks (Section 4.1), the fixed scale 448 of P-hat (Section 4.1)
and the mapping of query heads to KV heads under GQA (Algorithm 1's GQA note, Section 5.3).

Every expected value here is worked in NumPy (and torch's E4M3 cast, a library routine) from the
paper's definitions on operands built code by code; none comes from a second call of the oracle.
"""
import numpy as np
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

from test_oracle_formats import E2M1_MAG, e4m3_value

LOG2E = np.float32(1.4426950408889634)
UNIT = 0x38   # E4M3 code of 1.0


def _e2m1_vals(codes):
    """[..., 64] packed bytes -> [..., 128] FP64 values (even channel in the low nibble)."""
    tab = np.array(E2M1_MAG + [-m for m in E2M1_MAG], np.float64)
    return np.stack([tab[codes & 15], tab[codes >> 4]], axis=-1).reshape(*codes.shape[:-1], 128)


def _e4m3_vals(codes):
    return np.vectorize(lambda c: e4m3_value(int(c)))(codes).astype(np.float64)


def _e4m3_codes_rne(x32):
    """Round-to-nearest-even E4M3 codes of non-negative FP32 values <= 448 (library cast)."""
    return torch.from_numpy(np.ascontiguousarray(x32, np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()


def _two_block_case(seed=11, n_keys=256):
    """One head, one query row, unit block scales, so the logits are the plain dot products of the
    E2M1 values.  The key with the largest logit is placed in the second block and the first block
    is kept well below it, so the two traversal orders quantize the first block against different
    maxima."""
    rng = np.random.default_rng(seed)
    qc = rng.integers(0, 256, (1, 1, 1, 64), dtype=np.uint8)
    kc = rng.integers(0, 256, (1, 1, n_keys, 64), dtype=np.uint8)
    qv = _e2m1_vals(qc)[0, 0, 0]
    # key 200 = the query's own codes: its logit |q|^2 is the row maximum by a wide margin
    kc[0, 0, 200] = qc[0, 0, 0]
    s = _e2m1_vals(kc)[0, 0] @ qv
    assert s.argmax() == 200 and s[:128].max() < s[200] - 100
    vc = rng.integers(0, 256, (1, 1, n_keys, 128), dtype=np.uint8)
    vc[(vc & 0x7F) == 0x7F] = 0x10                      # no NaN patterns
    sf_q = np.full((1, 1, 1, 8), UNIT, np.uint8)
    sf_k = np.full((1, 1, n_keys, 8), UNIT, np.uint8)
    z = orc.Quantized(qc, sf_q, kc, sf_k, vc, None, None, None, np.ones(1, np.float32), np.ones(1, np.float32), 1.0)
    return z, s.astype(np.float32), _e4m3_vals(vc[0, 0]).astype(np.float32)


def _loop_by_hand(s, vd, lam, order, block=128):
    """Algorithm 1 lines 8-16 for one row, FP32 step by step, KV blocks in the given order.
    Returns the P-hat code of every key, the output row and (m, l)."""
    f32 = np.float32
    n = len(s)
    m, l = f32(-np.inf), f32(0)
    o = np.zeros(128, np.float32)
    codes = np.zeros(n, np.uint8)
    for jb in order:
        a, b = jb * block, min((jb + 1) * block, n)
        m_new = max(m, s[a:b].max())
        mlam = f32(m_new * lam)
        alpha = f32(0) if m == -np.inf else f32(np.exp2(np.float64(f32((m - m_new) * lam))))
        # P = 2^(lam S - lam m): the fused multiply-add is one rounding of the exact product minus mlam
        arg = (s[a:b].astype(np.float64) * np.float64(lam) - np.float64(mlam)).astype(np.float32)
        p = np.exp2(arg.astype(np.float64)).astype(np.float32)
        rs = f32(0)
        for x in p:                                       # l from the unquantized P, keys ascending
            rs = f32(rs + x)
        l = f32(f32(alpha * l) + rs)
        c = _e4m3_codes_rne(p * f32(448.0))               # fixed scale 448, no amax (Section 4.1)
        codes[a:b] = c
        ph = _e4m3_vals(c).astype(np.float32)
        acc = (alpha * o).astype(np.float32)
        for j in range(a, b):                             # keys ascending, FP32
            acc = (acc + ph[j - a] * vd[j]).astype(np.float32)
        o, m = acc, m_new
    out = (o / f32(f32(448.0) * l)).astype(np.float32)
    return codes, out, m, l


def test_reverse_traversal_is_what_the_loop_does():
    """Section 4.1: KV blocks are visited from the last to the first.  With the row maximum in the
    last block, the reverse order quantizes every P against the final maximum; the forward order
    quantizes the first block against its own, smaller maximum (its arg-max key gets 448) and
    rescales afterwards.  The oracle must produce the reverse pattern, and its forward switch the
    other one."""
    z, s, vd = _two_block_case()
    scale = 0.004      # the first block's keys keep weights comparable to the maximum's
    lam = np.float32(np.float32(np.float32(scale) * LOG2E) * np.float32(1.0)) * np.float32(1.0)
    rows = np.array([[0, 0, 0]], np.int32)
    want_rev, out_rev, m_rev, l_rev = _loop_by_hand(s, vd, lam, [1, 0])
    want_fwd, out_fwd, _, _ = _loop_by_hand(s, vd, lam, [0, 1])
    # the two orders differ where it matters: block 0's local arg-max has the top code only in forward order
    j0 = int(s[:128].argmax())
    assert want_fwd[j0] == 0x7E and want_rev[j0] < 0x7E
    assert (want_fwd[:128] != want_rev[:128]).sum() >= 10
    assert np.abs(out_fwd - out_rev).max() > 1e-4
    got_rev, ml = orc.phat_rows(z, rows, scale, False, reverse=True)
    got_fwd, _ = orc.phat_rows(z, rows, scale, False, reverse=False)
    assert np.array_equal(got_rev[0], want_rev)
    assert np.array_equal(got_fwd[0], want_fwd)
    assert ml[0, 0] == m_rev and abs(ml[0, 1] - l_rev) <= 1e-6 * l_rev
    o_rev, _ = orc.prefill_rows(z, rows, scale, False, reverse=True)
    o_fwd, _ = orc.prefill_rows(z, rows, scale, False, reverse=False)
    assert np.abs(o_rev[0] - out_rev).max() <= 1e-6
    assert np.abs(o_fwd[0] - out_fwd).max() <= 1e-6
    # the default of the front end is the paper's order
    o_def, _ = orc.prefill_rows(z, rows, scale, False)
    assert np.array_equal(o_def, o_rev) and not np.array_equal(o_def, o_fwd)


def test_traversal_order_changes_the_fp8_result():
    """With P in FP8 the order is part of the method: on a row whose large logits come late the two
    orders must not agree (they would only if the switch were ignored)."""
    w = wl.prefill_workload("t", 41, 1, 512, 1, 1, False)
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(1, 1, 64)
    a, _ = orc.prefill_rows(z, rows, w.softmax_scale, False, reverse=True)
    b, _ = orc.prefill_rows(z, rows, w.softmax_scale, False, reverse=False)
    assert np.abs(a - b).max() > 1e-4
    assert np.abs(a - b).mean() < 2e-2


def test_phat_uses_the_fixed_scale_448_and_the_subnormal_codes():
    """Section 4.1: P-hat = E4M3(448 P).  In the block where a row attains its final maximum the
    arg-max key has P = 1, i.e. code 0x7E; a row with a spread of logits reaches down into the
    subnormal codes 0x01..0x07 (448 P between 2^-10 and 2^-6) and to 0 below.  Every code equals
    the round-to-nearest-even image of 448 P worked in NumPy; a different scale (say 256 with the
    factor put back after decoding) gives other codes."""
    z, s, vd = _two_block_case()
    rows = np.array([[0, 0, 0]], np.int32)
    for scale in (0.0105, 0.006, 0.004):
        lam = np.float32(np.float32(scale) * LOG2E)
        got, _ = orc.phat_rows(z, rows, scale, False)
        want, out, _, _ = _loop_by_hand(s, vd, lam, [1, 0])
        assert np.array_equal(got[0], want)
        assert got[0, 200] == 0x7E and (got[0] == 0x7E).sum() == 1
        o, _ = orc.prefill_rows(z, rows, scale, False)
        assert np.abs(o[0] - out).max() <= 1e-6
        # direct statement for single keys: P = 2^(lam (s - M)), code = RNE_E4M3(448 P)
        M = s.max()
        for j in (0, 77, 128, 199, 201, 255):
            p = np.float32(np.exp2(np.float64(np.float32(np.float64(s[j]) * np.float64(lam) - np.float64(np.float32(M * lam))))))
            assert got[0, j] == int(_e4m3_codes_rne(np.array([p * np.float32(448.0)]))[0])
    # at this scale most keys sit 15 to 19 binades under the maximum: subnormal codes are in use, and so is 0
    got, _ = orc.phat_rows(z, rows, 0.0105, False)
    used = set(int(c) for c in got[0])
    assert used & set(range(1, 8)), used
    assert 0 in used


def _gqa_case():
    """H_q = 4, H_kv = 2, the two KV heads visibly different (their own offsets and their own V)."""
    w = wl.prefill_workload("gqa", 42, 1, 200, 4, 2, True, q_bias=True)
    k = w.k.clone().float()
    v = w.v.clone().float()
    k[:, :, 1] = -k[:, :, 1] + 3.0
    v[:, :, 1] = v[:, :, 1] * 0.25 + 5.0
    k = wl._finish(k)
    v = wl._finish(v)
    return w, orc.bf16_bits(w.q), orc.bf16_bits(k), orc.bf16_bits(v)


def test_means_are_per_head():
    """Eq. 7 with H > 1: one mean per (batch, head, channel), tokens summed in FP64."""
    w, q, k, v = _gqa_case()
    for x in (q, k):
        xf = orc.bits_to_f32(x).astype(np.float64)          # [B, N, H, 128]
        want = (xf.sum(axis=1) / x.shape[1]).astype(np.float32)
        got = orc.means(x)
        assert got.shape == (1, x.shape[2], 128)
        assert np.array_equal(got, want)
    km = orc.means(k)
    assert np.abs(km[0, 0] - km[0, 1]).max() > 1.0          # the heads really differ


def test_gqa_query_head_h_reads_kv_head_h_div_group():
    """Algorithm 1's GQA note: the G = H_q / H_kv query heads [g G, (g+1) G) share KV head g.
    Delta_S (Eq. 9), the logits (Eq. 10/11) and the outputs are recomputed in NumPy with hq // G."""
    w, q, k, v = _gqa_case()
    z = orc.stage1(q, k, v)
    Hq, Hkv, G, N = 4, 2, 2, 200
    kf = orc.bits_to_f32(k)
    dqk = float(z.dq[0]) * float(z.dk[0])
    qd = _e2m1_vals(z.q_codes) * np.repeat(_e4m3_vals(z.q_sf), 16, axis=-1)       # [1,4,N,128], MMA units
    kd = _e2m1_vals(z.k_codes) * np.repeat(_e4m3_vals(z.k_sf), 16, axis=-1)       # [1,2,N,128]
    vd = _e4m3_vals(z.v_codes)
    assert np.abs(vd[0, 0] - vd[0, 1]).mean() > 1.0
    rows = np.array([[0, h, i] for h in range(Hq) for i in (0, 5, 199)], np.int32)
    s_all = orc.logits_rows(z, rows)
    for hq in range(Hq):
        hk = hq // G
        kc32 = (kf[0, :, hk, :] - z.k_mean[0, hk]).astype(np.float64)
        want = (kc32 @ z.q_mean[0, hq].astype(np.float64)) / dqk
        want_bits = torch.from_numpy(want.astype(np.float32)).to(torch.bfloat16).view(torch.uint16).numpy()
        got_bits = z.delta[0, hq]
        ulp_off = np.abs(got_bits.astype(np.int64) - want_bits.astype(np.int64))
        assert ulp_off.max() <= 1 and (ulp_off == 0).mean() > 0.99
        # the other KV head would be far away
        other = ((kf[0, :, 1 - hk, :] - z.k_mean[0, 1 - hk]).astype(np.float64) @ z.q_mean[0, hq].astype(np.float64)) / dqk
        assert np.abs(other - want).mean() > 100 * np.abs(orc.bits_to_f32(got_bits) - want).mean()
        dl = orc.bits_to_f32(z.delta[0, hq]).astype(np.float64)
        for r, (_, h, i) in enumerate(rows):
            if h != hq:
                continue
            ref = kd[0, hk] @ qd[0, hq, i] + dl
            assert np.abs(s_all[r] - ref).max() <= 1e-6 * np.abs(ref).max()
            wrong = kd[0, 1 - hk] @ qd[0, hq, i] + dl
            assert np.abs(s_all[r] - wrong).max() > 1e-2 * np.abs(ref).max()
    # causal row 0 sees one key: the output is V-hat[hq // G][0] (P differs from 1 by at most the rounding of
    # lam*m inside the fused multiply-add, so l does too)
    r0 = np.array([[0, h, 0] for h in range(Hq)], np.int32)
    o32, _ = orc.prefill_rows(z, r0, w.softmax_scale, True)
    for hq in range(Hq):
        assert np.abs(o32[hq] - vd[0, hq // G, 0]).max() <= 4e-6
        assert np.abs(o32[hq] - vd[0, 1 - hq // G, 0]).max() > 1.0
    # decode with a one-token context: same statement through the decode entry point
    d32, _ = orc.decode(z.q_codes[:, :, 7], z.q_sf[:, :, 7], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0,
                        w.softmax_scale, np.array([1], np.int32))
    for hq in range(Hq):
        assert np.abs(d32[0, hq] - vd[0, hq // G, 0]).max() <= 4e-6
    # full rows against an FP64 recomputation with FP32 P (no code decisions involved): prefill and decode
    rows2 = np.array([[0, h, 150] for h in range(Hq)], np.int32)
    p32, _ = orc.prefill_rows(z, rows2, w.softmax_scale, True, p_fp8=False)
    dd32, _ = orc.decode(z.q_codes[:, :, 150], z.q_sf[:, :, 150], z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk,
                         1.0, w.softmax_scale, np.array([151], np.int32), p_fp8=False)
    lam = float(np.float32(w.softmax_scale)) * dqk
    for hq in range(Hq):
        hk = hq // G
        s = (kd[0, hk, :151] @ qd[0, hq, 150] + orc.bits_to_f32(z.delta[0, hq, :151]).astype(np.float64)) * lam
        p = np.exp(s - s.max())
        ref = (p / p.sum()) @ vd[0, hk, :151]
        assert np.abs(p32[hq] - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max())
        assert np.abs(dd32[0, hq] - ref).max() <= 2e-5 * max(1.0, np.abs(ref).max())
    # exact FP64 attention on the unquantized inputs maps heads the same way
    ex = orc.exact_rows(q, k, v, rows2, w.softmax_scale, True)
    qf, vf = orc.bits_to_f32(q).astype(np.float64), orc.bits_to_f32(v).astype(np.float64)
    for hq in range(Hq):
        hk = hq // G
        s = (kf[0, :151, hk].astype(np.float64) @ qf[0, 150, hq]) * float(np.float32(w.softmax_scale))
        p = np.exp(s - s.max())
        assert np.abs(ex[hq] - (p / p.sum()) @ vf[0, :151, hk]).max() < 1e-12


def test_eq8_identity_through_the_oracle():
    """Eq. 8-10 with the oracle's own Delta_S on one side: in true units,
    S_oracle(with Delta_S) - S_oracle(without) = Qbar . K_c up to the BF16 rounding of Delta_S, and adding the
    per-row constant Q . Kbar restores Q K^T up to the FP4 error of the centered products only."""
    w = wl.config1b_tiny_qbias()
    q, k, v = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    z = orc.stage1(q, k, v)
    rows = orc.all_rows(1, 1, 256)
    unit = float(z.dq[0]) * float(z.dk[0])
    s_with = orc.logits_rows(z, rows).astype(np.float64) * unit
    s_wo = orc.logits_rows(z, rows, use_delta=False).astype(np.float64) * unit
    Q = orc.bits_to_f32(q).astype(np.float64)[0, :, 0]
    K = orc.bits_to_f32(k).astype(np.float64)[0, :, 0]
    qb, kb = Q.mean(0), K.mean(0)
    Kc = K - kb
    comp = qb @ Kc.T                                         # second term of Eq. 8
    d = s_with - s_wo
    assert np.abs(d - comp[None, :]).max() <= (2.0 ** -8 + 1e-5) * np.abs(comp).max() + 1e-4
    assert np.abs(comp).max() > 5.0
    # first term of Eq. 8 from the quantized operands approximates Qc Kc^T; with the other two terms it is Q K^T
    S = Q @ K.T
    S_rebuilt = s_with + (Q @ kb)[:, None]
    S_no_comp = s_wo + (Q @ kb)[:, None]
    assert np.abs(S_rebuilt - S).mean() < 0.3 * np.abs(S_no_comp - S).mean()
    # the oracle's delta_s call alone against Eq. 9
    dl = orc.bits_to_f32(orc.delta_s(k, z.q_mean, z.k_mean, z.dq, z.dk, 1)[0, 0]).astype(np.float64) * unit
    assert np.abs(dl - comp).max() <= (2.0 ** -8 + 1e-5) * np.abs(comp).max() + 1e-4


def test_inspection_hooks_change_nothing_unless_asked():
    """The what-if hook of the inspection entry point (move one key's P-hat code by one step) is what the GPU tests
    use to show that a row outside the tolerance is a single code decision on a rounding boundary.  Without a flip
    it must reproduce the product function bit for bit; with one it must change exactly that code, and the output by
    that key's share: delta_code_value * (V_hat[k] - o) / (448 l) up to the rescaling roundings."""
    w = wl.prefill_workload("t", 5, 1, 300, 2, 1, True)
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    row = np.array([[0, 1, 200]], np.int32)
    ref, _ = orc.prefill_rows(z, row, w.softmax_scale, True)
    codes, ml, q, o = orc.phat_rows(z, row, w.softmax_scale, True, want_q=True)
    assert np.array_equal(o, ref)
    assert np.array_equal(_e4m3_codes_rne(q[0, :201]), codes[0, :201])
    key = int(np.argsort(q[0, :201])[-3])
    c2, _, _, o2 = orc.phat_rows(z, row, w.softmax_scale, True, want_q=True, flip_key=key, flip_dir=-1)
    diff = np.nonzero(c2[0] != codes[0])[0]
    assert list(diff) == [key] and int(c2[0, key]) == int(codes[0, key]) - 1
    dv = e4m3_value(int(c2[0, key])) - e4m3_value(int(codes[0, key]))
    vk = _e4m3_vals(z.v_codes[0, 0, key])
    # the key's share is dv * V_hat[k] / (448 l), scaled down by the alphas of the blocks visited after its own
    assert np.abs(o2[0] - o[0]).max() > 0
    assert np.abs(o2[0] - o[0]).max() <= np.abs(dv * vk / (448.0 * ml[0, 1])).max() * (1 + 1e-5) + 1e-7

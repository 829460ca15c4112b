"""Pins for the oracle's attention main loop (Algorithm 1 lines 6-20, Section 5.3)."""
import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

from test_oracle_formats import e4m3_value


def _np_softmax_attention(q, k, v, scale, n_vis):
    """Textbook softmax attention (Eq. 2) in FP64, row r sees keys [0, n_vis[r])."""
    out = np.zeros((q.shape[0], v.shape[1]))
    for r in range(q.shape[0]):
        n = n_vis[r]
        s = (k[:n] @ q[r]) * scale
        p = np.exp(s - s.max())
        out[r] = (p / p.sum()) @ v[:n]
    return out


@pytest.mark.parametrize("reverse", [True, False])
@pytest.mark.parametrize("block", [128, 64, 1000])
def test_mainloop_with_identity_quantizers_is_softmax_attention(reverse, block):
    rng = np.random.default_rng(5)
    q = rng.standard_normal((40, 128)).astype(np.float32)
    k = rng.standard_normal((700, 128)).astype(np.float32)
    v = rng.standard_normal((700, 128)).astype(np.float32)
    n_vis = np.array([1, 2, 127, 128, 129, 255, 256, 257, 640, 700] * 4, np.int32)
    out, rs = orc.mainloop_identity(q, k, v, n_vis, 1 / np.sqrt(128), block, reverse)
    ref = _np_softmax_attention(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64),
                                1 / np.sqrt(128), n_vis)
    assert np.max(np.abs(out - ref)) < 2e-6
    # rows of P / l sum to one
    assert np.max(np.abs(rs - 1.0)) < 1e-6


def test_traversal_order_only_changes_rounding():
    rng = np.random.default_rng(6)
    q = rng.standard_normal((8, 128)).astype(np.float32) * 3   # peaky rows
    k = rng.standard_normal((512, 128)).astype(np.float32)
    v = rng.standard_normal((512, 128)).astype(np.float32)
    n_vis = np.full(8, 512, np.int32)
    a, _ = orc.mainloop_identity(q, k, v, n_vis, 1 / np.sqrt(128), 128, True)
    b, _ = orc.mainloop_identity(q, k, v, n_vis, 1 / np.sqrt(128), 128, False)
    # FP32 P: the two orders are the same sum in another order, so they differ, but only by rounding
    assert 0 < np.max(np.abs(a - b)) < 2e-6


def _stage1(w, **kw):
    return orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v), **kw)


def test_logits_with_unit_scales_equal_integer_dot():
    # Eq. 10 with all block scales 1 and no compensation is an integer dot product of (codes x 2)
    rng = np.random.default_rng(7)
    qc = rng.integers(0, 256, (1, 1, 4, 64), dtype=np.uint8)
    kc = rng.integers(0, 256, (1, 1, 300, 64), dtype=np.uint8)
    one = np.full((1, 1, 4, 8), 0x38, np.uint8)
    onek = np.full((1, 1, 300, 8), 0x38, np.uint8)
    z = orc.Quantized(qc, one, kc, onek, np.zeros((1, 1, 300, 128), np.uint8), None, None, None,
                      np.ones(1, np.float32), np.ones(1, np.float32), 1.0)
    rows = orc.all_rows(1, 1, 4)
    s = orc.logits_rows(z, rows, use_delta=False)
    twice = np.array([0, 1, 2, 3, 4, 6, 8, 12, 0, -1, -2, -3, -4, -6, -8, -12], np.int64)

    def unpack(c):
        return np.stack([twice[c & 15], twice[c >> 4]], axis=-1).reshape(*c.shape[:-1], 128)

    ref = unpack(qc)[0, 0] @ unpack(kc)[0, 0].T
    assert np.array_equal(s.astype(np.float64) * 4, ref.astype(np.float64))


def test_logits_apply_block_scales_and_seed():
    w = wl.config1b_tiny_qbias()
    z = _stage1(w)
    rows = np.array([[0, 0, 3], [0, 0, 200]], np.int32)
    s = orc.logits_rows(z, rows)
    # independent FP64 recomputation from the decoded operands
    from test_oracle_stage1 import _dequant
    qd = _dequant(z.q_codes, z.q_sf, np.ones(1, np.float32)).astype(np.float64)[0, 0]
    kd = _dequant(z.k_codes, z.k_sf, np.ones(1, np.float32)).astype(np.float64)[0, 0]
    dl = orc.bits_to_f32(z.delta[0, 0]).astype(np.float64)
    ref = qd[[3, 200]] @ kd.T + dl[None, :]
    assert np.max(np.abs(s - ref)) <= 1e-6 * np.max(np.abs(ref))
    # and the compensated logits, put back in true units, track the true logits Q K^T minus the
    # per-row constant (Q Kbar^T), which softmax ignores (Eq. 8-10)
    Q = w.q.double()[0, :, 0, :].numpy()
    K = w.k.double()[0, :, 0, :].numpy()
    true = Q[[3, 200]] @ K.T - (Q[[3, 200]] @ z.k_mean[0, 0].astype(np.float64))[:, None]
    approx = s.astype(np.float64) * float(z.dq[0]) * float(z.dk[0])
    no_comp = orc.logits_rows(z, rows, use_delta=False).astype(np.float64) * float(z.dq[0]) * float(z.dk[0])
    assert np.abs(approx - true).mean() < 0.25 * np.abs(no_comp - true).mean()


def test_single_key_row_returns_dequantized_v():
    # causal row 0 sees one key: P = 1 -> P_hat = 448 exactly -> O = V_hat[0]
    w = wl.prefill_workload("t", 31, 1, 128, 2, 1, True)
    z = _stage1(w)
    rows = np.array([[0, 0, 0], [0, 1, 0]], np.int32)
    o32, o16 = orc.prefill_rows(z, rows, w.softmax_scale, True)
    v0 = np.array([e4m3_value(int(c)) for c in z.v_codes[0, 0, 0]], np.float32)
    assert np.array_equal(o32[0], v0) and np.array_equal(o32[1], v0)
    assert np.array_equal(orc.bits_to_f32(o16[0]), v0)  # E4M3 values are exact in BF16


def test_qk4pv8_tracks_exact_attention_and_compensation_helps():
    w = wl.config1b_tiny_qbias()
    z = _stage1(w)
    rows = orc.all_rows(1, 1, 256)
    q, k, v = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    exact = orc.exact_rows(q, k, v, rows, w.softmax_scale, False)
    with_c, _ = orc.prefill_rows(z, rows, w.softmax_scale, False)
    no_c, _ = orc.prefill_rows(z, rows, w.softmax_scale, False, use_delta=False)
    e_with = np.abs(with_c - exact).mean()
    e_without = np.abs(no_c - exact).mean()
    assert e_with < 0.1
    assert e_with < 0.5 * e_without
    # exact attention itself: compare the FP64 C routine with numpy
    ref = _np_softmax_attention(w.q.double()[0, :, 0].numpy(), w.k.double()[0, :, 0].numpy(),
                                w.v.double()[0, :, 0].numpy(), float(np.float32(w.softmax_scale)), [256] * 256)
    assert np.max(np.abs(exact - ref)) < 1e-12


def test_fp8_p_is_the_only_difference_to_fp32_p():
    w = wl.config1_tiny()
    z = _stage1(w)
    rows = orc.all_rows(1, 1, 256)
    a, _ = orc.prefill_rows(z, rows, w.softmax_scale, False, p_fp8=True)
    b, _ = orc.prefill_rows(z, rows, w.softmax_scale, False, p_fp8=False)
    d = np.abs(a - b)
    assert 0 < d.mean() < 2e-2      # E4M3 has 3 mantissa bits: a few percent per term, averaged down
    assert np.isfinite(a).all()


def test_causal_mask_bottom_right_alignment():
    # N_q < N_kv: query i sees keys up to i + N_kv - N_q
    w = wl.prefill_workload("t", 32, 1, 384, 1, 1, True, N_q=130)
    z = _stage1(w)
    rows = np.array([[0, 0, 0], [0, 0, 129]], np.int32)
    o, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    # same rows computed non-causally on truncated keys
    import copy
    for r, n in ((0, 255), (1, 384)):
        zt = copy.copy(z)
        zt.k_codes, zt.k_sf = z.k_codes[:, :, :n].copy(), z.k_sf[:, :, :n].copy()
        zt.v_codes, zt.delta = z.v_codes[:, :, :n].copy(), z.delta[:, :, :n].copy()
        ot, _ = orc.prefill_rows(zt, rows[r:r + 1], w.softmax_scale, False)
        assert np.array_equal(ot[0], o[r])


def test_decode_single_split_equals_prefill_row_and_merge_is_lse():
    w = wl.prefill_workload("t", 33, 1, 3000, 4, 2, False, N_q=1)
    z = _stage1(w)
    rows = orc.all_rows(1, 4, 1)
    qc, qs = z.q_codes[:, :, 0, :], z.q_sf[:, :, 0, :]
    seq = np.array([900], np.int32)
    # <= 1024 keys: one partition, must be bit-identical to the prefill main loop on the same keys
    import copy
    zt = copy.copy(z)
    zt.k_codes, zt.k_sf = z.k_codes[:, :, :900].copy(), z.k_sf[:, :, :900].copy()
    zt.v_codes, zt.delta = z.v_codes[:, :, :900].copy(), z.delta[:, :, :900].copy()
    p32, _ = orc.prefill_rows(zt, rows, w.softmax_scale, False)
    d32, d16 = orc.decode(qc, qs, z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0, w.softmax_scale, seq)
    assert np.array_equal(d32[0], p32)
    # 3000 keys = 3 partitions.  With FP32 P the partition/merge is plain log-sum-exp algebra and
    # must agree with the unpartitioned loop to rounding.
    seq = np.array([3000], np.int32)
    a, _ = orc.decode(qc, qs, z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0, w.softmax_scale, seq,
                      p_fp8=False)
    b, _ = orc.prefill_rows(z, rows, w.softmax_scale, False, p_fp8=False)
    assert np.max(np.abs(a[0] - b)) < 2e-6
    # with FP8 P the partitioning changes which running maximum each P is quantized against: close, not equal
    c, _ = orc.decode(qc, qs, z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0, w.softmax_scale, seq)
    e, _ = orc.prefill_rows(z, rows, w.softmax_scale, False)
    assert np.max(np.abs(c[0] - e)) < 0.1
    # empty request
    z0, _ = orc.decode(qc, qs, z.k_codes, z.k_sf, z.v_codes, z.delta, z.dq, z.dk, 1.0, w.softmax_scale,
                       np.array([0], np.int32))
    assert not z0.any()


def test_elementwise_placement_adds_the_same_term_after_the_products():
    """Section 7.4 (compensation placement): the ablation variant adds Delta_S to the finished FP32 score instead of
    seeding the accumulator with it.  Pinned against an FP64 recomputation from the decoded operands (a dropped
    term or a wrong sign would be off by the size of Delta_S itself), against the seeded placement (same term: only
    rounding-level differences), and without Delta_S the two must be the same function."""
    from test_oracle_stage1 import _dequant
    w = wl.config1b_tiny_qbias()
    z = _stage1(w)
    rows = np.array([[0, 0, 0], [0, 0, 3], [0, 0, 127], [0, 0, 128], [0, 0, 255]], np.int32)
    ew32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True, p_fp8=False, elementwise=True)
    qd = _dequant(z.q_codes, z.q_sf, np.ones(1, np.float32)).astype(np.float64)[0, 0]
    kd = _dequant(z.k_codes, z.k_sf, np.ones(1, np.float32)).astype(np.float64)[0, 0]
    dl = orc.bits_to_f32(z.delta[0, 0]).astype(np.float64)
    vd = np.vectorize(lambda c: e4m3_value(int(c)))(z.v_codes[0, 0]).astype(np.float64)
    lam = float(np.float32(w.softmax_scale)) * float(z.dq[0]) * float(z.dk[0])
    assert np.abs(dl).max() * lam > 0.5            # the term matters in this workload
    for r, i in enumerate(rows[:, 2]):
        s = (kd[:i + 1] @ qd[i] + dl[:i + 1]) * lam
        p = np.exp(s - s.max())
        ref = (p / p.sum()) @ vd[:i + 1]
        assert np.max(np.abs(ew32[r] - ref)) <= 2e-5 * max(1.0, np.abs(ref).max()), i
    all_rows = orc.all_rows(1, 1, 256)
    seeded, _ = orc.prefill_rows(z, all_rows, w.softmax_scale, True)
    added, _ = orc.prefill_rows(z, all_rows, w.softmax_scale, True, elementwise=True)
    d = np.abs(seeded - added)
    assert d.mean() < 1e-4 and d.max() < 0.05     # an FP32 rounding of S can flip an E4M3 code of P now and then
    a, _ = orc.prefill_rows(z, all_rows, w.softmax_scale, True, use_delta=False)
    b, _ = orc.prefill_rows(z, all_rows, w.softmax_scale, True, use_delta=False, elementwise=True)
    assert np.array_equal(a, b)


def test_bf16_pv_variant_against_fp64_recomputation():
    """Section 3.1's NVFP4 + BF16 assignment: same logits as the method, P in BF16, V unquantized BF16.  Pinned
    against an FP64 softmax over the oracle's own logits with the BF16 inputs of V (what is left is the BF16 rounding
    of P: 2^-9 relative per term, and FP32 summation), on GQA heads with visibly different V, and against the method:
    the two differ (FP8 P and FP8 V against BF16) but track each other."""
    from test_oracle_stage1 import _dequant
    w = wl.prefill_workload("t", 36, 1, 300, 4, 2, True, q_bias=True)
    v = w.v.clone().float()
    v[:, :, 1] = v[:, :, 1] * 0.5 + 3.0
    w.v = wl._finish(v)
    q, k, vb = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    z = orc.stage1(q, k, vb)
    rows = np.array([[0, h, i] for h in range(4) for i in (0, 127, 128, 299)], np.int32)
    o32, o16 = orc.prefill_rows_pv_bf16(z, vb, rows, w.softmax_scale, True)
    s = orc.logits_rows(z, rows).astype(np.float64)
    lam = float(np.float32(w.softmax_scale)) * float(z.dq[0]) * float(z.dk[0])
    vf = orc.bits_to_f32(vb).astype(np.float64)
    for r, (_, h, i) in enumerate(rows):
        x = s[r, :i + 1] * lam
        p = np.exp(x - x.max())
        ref = (p / p.sum()) @ vf[0, :i + 1, h // 2]
        assert np.abs(o32[r] - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-5, (h, i)
        wrong = (p / p.sum()) @ vf[0, :i + 1, 1 - h // 2]
        assert np.abs(o32[r] - wrong).max() > 0.5
    assert np.array_equal(o16, torch.from_numpy(o32).to(torch.bfloat16).view(torch.uint16).numpy())
    m32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    d = np.abs(m32 - o32)
    assert 1e-4 < d.mean() < 0.1
    # single-key rows return V itself (P = 1 up to the rounding of lam * m inside the fused multiply-add)
    assert np.abs(o32[0] - vf[0, 0, 0]).max() <= 1e-5

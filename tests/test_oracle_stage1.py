"""Pins for the oracle's statistics and quantizers (Algorithm 1 lines 1-5)."""
import numpy as np
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

from test_oracle_formats import E2M1_MAG, e4m3_value


def _cfg1():
    w = wl.config1_tiny()
    return w, orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)


def test_generator_shapes_and_flush():
    w, q, k, v = _cfg1()
    assert w.q.shape == (1, 256, 1, 128) and w.k.shape == (1, 256, 1, 128)
    for t in (w.q, w.k, w.v):
        a = t.float().abs()
        assert float(a[a > 0].min()) >= 2.0 ** -14
    # K carries the channel structure (offsets, outliers); Q and V do not
    assert float(w.k.float().mean(dim=1).abs().max()) > 1.0
    assert float(w.q.float().mean(dim=1).abs().max()) < 0.5
    # deterministic
    w2 = wl.config1_tiny()
    assert torch.equal(w.k, w2.k)


def test_means_exact_against_fixed_point():
    w = wl.prefill_workload("t", 77, 2, 1000, 3, 1, True)
    x = orc.bf16_bits(w.k)
    mean = orc.means(x)
    fixed = orc.colsum_fixed(x)      # exact integer sums in units of 2^-40
    ref = (fixed.astype(np.float64) * 2.0 ** -40 / 1000.0).astype(np.float32)
    # int64 -> float64 is exact here (|sum| < 2^13 in units needing < 53 bits)
    assert np.all(np.abs(fixed) < 2 ** 53)
    assert np.array_equal(mean, ref)
    # any summation order gives the same FP64 sum: compare with numpy's pairwise sum
    xf = orc.bits_to_f32(x).astype(np.float64)
    assert np.array_equal(mean, (xf.sum(axis=1) / 1000.0).astype(np.float32))
    assert np.array_equal(mean, (xf[:, ::-1].sum(axis=1) / 1000.0).astype(np.float32))


def _bf16(x):
    return torch.tensor(x, dtype=torch.float32).to(torch.bfloat16)


def test_worked_block_follows_tie_table():
    # A tensor whose centered amax is 2688 has d = 1, so a block with amax 6 gets
    # scale code 0x38 (1.0) and its elements land on the E2M1 grid literally.
    x = torch.zeros(1, 2, 1, 128, dtype=torch.bfloat16)
    vals = [6.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0, 0.0]
    x[0, 0, 0, :16] = _bf16(vals)
    x[0, 0, 0, 16] = 2688.0
    x[0, 0, 0, 32:48] = _bf16([3.0] + [0.0] * 15)    # amax 3 -> scale 0.5 -> 3/0.5 = 6
    bits = orc.bf16_bits(x)
    mean = np.zeros((1, 1, 128), np.float32)
    d = orc.tensor_scale(bits, mean)
    assert d[0] == 1.0
    codes, sf = orc.quantize_nvfp4(bits, mean, d)
    assert sf[0, 0, 0, 0] == 0x38 and sf[0, 0, 0, 1] == 0x7E and sf[0, 0, 0, 2] == 0x30
    got = []
    for i in range(8):
        byte = int(codes[0, 0, 0, i])
        got += [orc.e2m1_decode(byte & 15), orc.e2m1_decode(byte >> 4)]
    want = [6.0, 0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0, -0.0, -1.0, -1.0, -2.0, -2.0, -4.0, -4.0, 0.0]
    assert got == want
    assert int(codes[0, 0, 0, 4]) & 15 == 8          # -0.25 rounds to zero but keeps its sign bit
    assert int(codes[0, 0, 0, 8]) & 15 == 7          # 2688 / 448 = 6
    assert int(codes[0, 0, 0, 16]) & 15 == 7         # 3 / 0.5 = 6
    # token 1 is all zeros: scale code 0, all codes 0
    assert not sf[0, 0, 1].any() and not codes[0, 0, 1].any()


def _dequant(codes, sf, d):
    lo = np.vectorize(lambda c: orc.e2m1_decode(int(c) & 15))(codes).astype(np.float32)
    hi = np.vectorize(lambda c: orc.e2m1_decode(int(c) >> 4))(codes).astype(np.float32)
    vals = np.stack([lo, hi], axis=-1).reshape(*codes.shape[:-1], 128)
    s = np.vectorize(lambda c: e4m3_value(int(c)))(sf).astype(np.float32)
    return vals * np.repeat(s, 16, axis=-1) * d.reshape(-1, 1, 1, 1)


def test_quantizer_invariants_config1():
    w, q, k, v = _cfg1()
    z = orc.stage1(q, k, v)
    # per-tensor scale: the block holding the tensor maximum gets the largest scale code
    assert z.k_sf.max() == 0x7E and z.q_sf.max() == 0x7E
    assert not (z.k_sf & 0x80).any()
    # every block with a normal, unsaturated scale contains a magnitude-6 code
    for codes, sf in ((z.k_codes, z.k_sf), (z.q_codes, z.q_sf)):
        mag = np.maximum(codes & 7, (codes >> 4) & 7).reshape(*sf.shape, 8).max(axis=-1)
        sel = (sf >= 0x08) & (sf < 0x7E)
        assert sel.sum() > 100
        assert np.all(mag[sel] == 7)
    # reconstruction error of Eq. 1: at most half an E2M1 step (1.0 at the top of the grid) times the scale,
    # plus the saturation of elements between 6 s and amax when the scale rounded down
    kc = orc.bits_to_f32(k).transpose(0, 2, 1, 3) - z.k_mean[:, :, None, :]
    deq = _dequant(z.k_codes, z.k_sf, z.dk)
    s = np.repeat(np.vectorize(lambda c: e4m3_value(int(c)))(z.k_sf), 16, axis=-1) * z.dk[0]
    assert np.all(np.abs(deq - kc) <= 1.0 * s * (1 + 1e-6) + 1e-12)
    assert np.mean(np.abs(deq - kc)) < 0.12 * np.mean(np.abs(kc))


def test_centering_shrinks_blocks_with_channel_offsets():
    # Section 4.2: removing the per-channel mean lowers the K quantization error
    w, q, k, v = _cfg1()
    zs = orc.stage1(q, k, v, smooth=True)
    zd = orc.stage1(q, k, v, smooth=False)
    kf = orc.bits_to_f32(k).transpose(0, 2, 1, 3)
    err_s = np.abs(_dequant(zs.k_codes, zs.k_sf, zs.dk) + zs.k_mean[:, :, None, :] - kf).mean()
    err_d = np.abs(_dequant(zd.k_codes, zd.k_sf, zd.dk) - kf).mean()
    assert err_s < 0.8 * err_d
    assert zd.delta is None and not zd.k_mean.any()


def test_v_codes_match_torch_cast_and_roundtrip():
    w, q, k, v = _cfg1()
    vc = orc.quantize_v(v, 1.0)
    ref = w.v.float().to(torch.float8_e4m3fn).view(torch.uint8).permute(0, 2, 1, 3).numpy()
    assert np.array_equal(vc, ref)
    # BF16 values that are exactly E4M3 values survive unchanged
    exact = torch.tensor([[e4m3_value(c) for c in range(0, 127)] + [0.0]], dtype=torch.float32)
    x = exact.to(torch.bfloat16).view(1, 1, 1, 128)
    vc = orc.quantize_v(orc.bf16_bits(x), 1.0)
    assert list(vc[0, 0, 0, :127]) == list(range(127))
    # saturation, never NaN
    big = torch.full((1, 1, 1, 128), 1000.0, dtype=torch.bfloat16)
    big[..., 1] = -1000.0
    vc = orc.quantize_v(orc.bf16_bits(big), 1.0)
    assert vc[0, 0, 0, 0] == 0x7E and vc[0, 0, 0, 1] == 0xFE
    # optional scale
    vc2 = orc.quantize_v(orc.bf16_bits(big), 4.0)
    assert e4m3_value(int(vc2[0, 0, 0, 0])) == 256.0  # 250 rounds to 256 (neighbours 240 and 256)


def test_delta_s_definition_and_bf16_bound():
    w = wl.config1b_tiny_qbias()
    q, k, v = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    z = orc.stage1(q, k, v)
    kc = orc.bits_to_f32(k).astype(np.float64)[0, :, 0, :] - z.k_mean[0, 0].astype(np.float64)
    # centering itself is one FP32 rounding; redo it in FP32 for the exact comparison
    kc32 = (orc.bits_to_f32(k)[0, :, 0, :] - z.k_mean[0, 0]).astype(np.float64)
    want = kc32 @ z.q_mean[0, 0].astype(np.float64) / (float(z.dq[0]) * float(z.dk[0]))
    got = orc.bits_to_f32(z.delta[0, 0]).astype(np.float64)
    # one BF16 rounding: relative error at most 2^-8 (Section 4.3), plus the FP32 step before it
    assert np.all(np.abs(got - want) <= np.abs(want) * (2.0 ** -8 + 2.0 ** -22) + 1e-30)
    assert np.abs(want).max() > 10 * 2.0 ** -8      # the vector is far from zero here
    assert np.allclose(kc, kc32, atol=1e-5)


def test_eq8_decomposition_identity_fp64():
    # S = Qc Kc^T + 1 (Qbar Kc^T) + (Q Kbar^T) 1^T, and the last term cancels under softmax
    w = wl.config1b_tiny_qbias()
    Q = w.q.double()[0, :, 0, :].numpy()
    K = w.k.double()[0, :, 0, :].numpy()
    qb, kb = Q.mean(0), K.mean(0)
    Qc, Kc = Q - qb, K - kb
    S = Q @ K.T
    S2 = Qc @ Kc.T + np.outer(np.ones(len(Q)), qb @ Kc.T) + np.outer(Q @ kb, np.ones(len(K)))
    assert np.max(np.abs(S - S2)) <= 1e-12 * np.max(np.abs(S))

    def softmax(x):
        e = np.exp(x - x.max(axis=1, keepdims=True))
        return e / e.sum(axis=1, keepdims=True)

    P = softmax(S / np.sqrt(128))
    P2 = softmax((Qc @ Kc.T + np.outer(np.ones(len(Q)), qb @ Kc.T)) / np.sqrt(128))
    assert np.max(np.abs(P - P2)) < 1e-12

"""Pins for the oracle's statement of the NVFP4 + NVFP4 precision assignment (Section 3.1, Section 7.2):
the V quantizer with its 16-element blocks along the token axis, and the attention loop whose P enters
the second MMA as a block-scaled E2M1 operand.

Every expected value is worked in NumPy (nearest-value search over the E2M1 table, torch's E4M3 cast as
the library routine for the block scales) from the definitions; none comes from a second call of the oracle.
"""
import numpy as np
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

from test_oracle_formats import E2M1_MAG
from test_oracle_semantics import LOG2E, UNIT, _e2m1_vals, _e4m3_codes_rne, _e4m3_vals

MAG = np.array(E2M1_MAG, np.float64)


def _e2m1_codes_rne(y32):
    """Nearest E2M1 code of FP32 values (brute force over the eight magnitudes, ties to the even code,
    saturating, sign in bit 3)."""
    y = np.asarray(y32, np.float32)
    a = np.abs(y).astype(np.float64)
    dist = np.abs(a[..., None] - MAG)                                    # [..., 8]
    best = dist.min(axis=-1, keepdims=True)
    cand = dist == best
    even_first = np.where(cand & (np.arange(8) % 2 == 0), np.arange(8), 99).min(axis=-1)
    any_first = np.where(cand, np.arange(8), 99).min(axis=-1)
    code = np.where(even_first < 99, even_first, any_first).astype(np.uint8)
    return code | (np.signbit(y).astype(np.uint8) << 3)


def _signed_vals(codes4):
    return np.where(codes4 & 8, -MAG[codes4 & 7], MAG[codes4 & 7])


def _quantize_v_by_hand(v_bits, d):
    """Eq. 1 with the blocks along the token axis: returns codes [B,H,128,NB,16] (one per token) and sf [B,H,128,NB]."""
    f32 = np.float32
    x = orc.bits_to_f32(v_bits)                                          # [B,N,H,128]
    B, N, H, _ = x.shape
    NB = (N + 15) // 16
    xp = np.zeros((B, NB * 16, H, 128), np.float32)
    xp[:, :N] = x
    xb = xp.transpose(0, 2, 3, 1).reshape(B, H, 128, NB, 16)             # [B,H,c,blk,16]
    amax = np.abs(xb).max(axis=-1)
    r = (amax / f32(f32(6.0) * f32(d))).astype(np.float32)
    sc = _e4m3_codes_rne(r)
    s = (_e4m3_vals(sc).astype(np.float32) * f32(d)).astype(np.float32)
    with np.errstate(divide="ignore"):
        inv = (f32(1.0) / s).astype(np.float32)
    inv[~(s > 0) | np.isinf(inv)] = 0
    y = (xb * inv[..., None]).astype(np.float32)
    return _e2m1_codes_rne(y), sc


def _unpack(codes8):
    """[..., 8] bytes -> [..., 16] codes, the even element in the low nibble."""
    return np.stack([codes8 & 15, codes8 >> 4], axis=-1).reshape(*codes8.shape[:-1], 16)


def test_v_quantizer_blocks_lie_along_the_token_axis():
    """A ragged length (2.5 blocks), two heads: codes and scales equal the NumPy statement; a quantizer with its
    blocks along the channel axis (the Q/K one) or with the heads swapped gives other bytes."""
    w = wl.prefill_workload("t", 5, 2, 40, 2, 2, False)
    v = orc.bf16_bits(w.v)
    d = float(np.float32(np.abs(orc.bits_to_f32(v)).max() / (6.0 * 448.0)))
    codes, sf = orc.quantize_v_fp4(v, d)
    want_c, want_s = _quantize_v_by_hand(v, d)
    assert sf.shape == (2, 2, 128, 3) and codes.shape == (2, 2, 128, 3, 8)
    assert np.array_equal(sf, want_s)
    assert np.array_equal(_unpack(codes), want_c)
    # the tail of the last block (tokens 40..47) is zero
    assert (_unpack(codes)[:, :, :, 2, 8:] & 7).max() == 0
    # blocks along the wrong axis: the Q/K quantizer on the same tensor has other scales
    zc, zs = orc.quantize_nvfp4(v, np.zeros((2, 2, 128), np.float32), np.full(2, d, np.float32))
    assert zs.shape == (2, 2, 40, 8)
    # and the heads are where they belong
    assert not np.array_equal(sf[:, 0], sf[:, 1])
    x = orc.bits_to_f32(v)
    deq = _signed_vals(_unpack(codes)) * (_e4m3_vals(sf)[..., None] * d)              # [B,H,128,NB,16]
    deq = deq.reshape(2, 2, 128, 48)[..., :40].transpose(0, 3, 1, 2)
    err = np.abs(deq - x)
    assert err.mean() < 0.1 * np.abs(x).mean()                                         # it is V, coarsely
    assert err.max() <= np.abs(x).max() / 6 + 1e-6                                     # half of the largest E2M1 step 2 * scale


def test_v_quantizer_reproduces_values_built_from_codes():
    """A tensor built as code x scale x d, every block containing a 6, comes back code for code."""
    rng = np.random.default_rng(3)
    B, N, H = 1, 64, 1
    d = 2.0 ** -7
    c4 = rng.integers(0, 16, (B, H, 128, 4, 16), dtype=np.uint8)
    c4[..., 0] = 7                                                        # +6 in every block
    c4[(c4 & 7) == 0] = 0                                                 # no negative zeros
    sc = rng.integers(0x28, 0x48, (B, H, 128, 4), dtype=np.uint8)          # normal scales close to 1.0
    x = _signed_vals(c4) * (_e4m3_vals(sc)[..., None] * d)                # exact in BF16: <= 2+4 significant bits
    x = x.reshape(B, H, 128, N).transpose(0, 3, 1, 2).astype(np.float32)
    bits = (np.ascontiguousarray(x).view(np.uint32) >> 16).astype(np.uint16)
    assert np.array_equal(orc.bits_to_f32(bits), x)
    codes, sf = orc.quantize_v_fp4(bits, d)
    assert np.array_equal(sf, sc)
    assert np.array_equal(_unpack(codes), c4)


def _case(seed=17, n_keys=200):
    """One head, one query row, unit Q/K block scales (logits = plain dot products of E2M1 values), the row maximum
    in the second KV block, a BF16 V."""
    rng = np.random.default_rng(seed)
    qc = rng.integers(0, 256, (1, 1, 1, 64), dtype=np.uint8)
    kc = rng.integers(0, 256, (1, 1, n_keys, 64), dtype=np.uint8)
    kc[0, 0, 150] = qc[0, 0, 0]
    qv = _e2m1_vals(qc)[0, 0, 0]
    s = (_e2m1_vals(kc)[0, 0] @ qv).astype(np.float32)
    assert s.argmax() == 150
    v = torch.from_numpy(rng.standard_normal((1, n_keys, 1, 128)).astype(np.float32)).to(torch.bfloat16)
    vb = orc.bf16_bits(v)
    sf_q = np.full((1, 1, 1, 8), UNIT, np.uint8)
    sf_k = np.full((1, 1, n_keys, 8), UNIT, np.uint8)
    z = orc.Quantized(qc, sf_q, kc, sf_k, np.zeros((1, 1, n_keys, 128), np.uint8), None, None, None,
                      np.ones(1, np.float32), np.ones(1, np.float32), 1.0)
    return z, s, vb


def _loop_by_hand(s, vcode, vsf, d_v, lam, block=128):
    """The assignment's loop for one row in FP32, step by step; KV blocks last to first.
    vcode [128, NB, 16] E2M1 codes, vsf [128, NB] E4M3 codes."""
    f32 = np.float32
    n = len(s)
    NB = vsf.shape[1]
    m, l = f32(-np.inf), f32(0)
    o = np.zeros(128, np.float32)
    pcodes = np.zeros(NB * 16, np.uint8)
    psf = np.zeros(NB, np.uint8)
    vval = _signed_vals(vcode).astype(np.float32)
    vscale = _e4m3_vals(vsf).astype(np.float32)
    for jb in range((n - 1) // block, -1, -1):
        a, b = jb * block, min((jb + 1) * block, n)
        m_new = max(m, s[a:b].max())
        mlam = f32(m_new * lam)
        alpha = f32(0) if m == -np.inf else f32(np.exp2(np.float64(f32((m - m_new) * lam))))
        arg = (s[a:b].astype(np.float64) * np.float64(lam) - np.float64(mlam)).astype(np.float32)
        p = np.exp2(arg.astype(np.float64)).astype(np.float32)
        rs = f32(0)
        for x in p:
            rs = f32(rs + x)
        l = f32(f32(alpha * l) + rs)
        q = np.zeros(-(-(b - a) // 16) * 16, np.float32)
        q[: b - a] = p * f32(448.0)
        acc = (alpha * o).astype(np.float32)
        for g in range(len(q) // 16):
            blk = q[16 * g: 16 * g + 16]
            sc = _e4m3_codes_rne(np.array([blk.max()], np.float32))[0]
            sp = f32(_e4m3_vals(np.array([sc]))[0])
            inv = f32(6.0) / sp if sp > 0 else f32(0)
            code = _e2m1_codes_rne((blk * inv).astype(np.float32))
            gi = a // 16 + g
            pcodes[16 * gi: 16 * gi + 16] = code
            psf[gi] = sc
            dot = (MAG[code & 7].astype(np.float32)[None, :] * vval[:, gi, :]).sum(axis=1, dtype=np.float64)   # exact
            acc = (acc + (sp * vscale[:, gi]).astype(np.float32) * dot.astype(np.float32)).astype(np.float32)
        o, m = acc, m_new
    out = (o / f32(f32(2688.0) * l) * f32(d_v)).astype(np.float32)
    return pcodes[:n], psf, out


def test_fp4_pv_loop_against_the_numpy_statement():
    """Two KV blocks, ragged second one; three softmax scales from peaked to flat.  Codes and block scales of P
    bit for bit, the output to FP32 rounding."""
    z, s, vb = _case()
    d_v = float(np.float32(np.abs(orc.bits_to_f32(vb)).max() / (6.0 * 448.0)))
    vc, vs = orc.quantize_v_fp4(vb, d_v)
    rows = np.array([[0, 0, 0]], np.int32)
    for scale in (0.02, 0.006, 0.002):
        lam = np.float32(np.float32(scale) * LOG2E)
        want_c, want_s, want_o = _loop_by_hand(s, _unpack(vc[0, 0]), vs[0, 0], d_v, lam)
        o32, _, pc, ps, _, _ = orc.prefill_rows_pv_fp4(z, vc, vs, d_v, rows, scale, False, want_codes=True)
        assert np.array_equal(pc[0], want_c), scale
        assert np.array_equal(ps[0], want_s), scale
        assert np.abs(o32[0] - want_o).max() <= 2e-6 * max(1.0, np.abs(want_o).max()), scale
        # the block that holds the row maximum has scale code 0x7E (max q = 448) and its arg-max key the code of 6
        assert want_s[150 // 16] == 0x7E and want_c[150] == 7
    # flat enough that blocks of the first KV block carry weight too: their scales are below the top one and non-zero
    assert 0 < want_s[:8].max() < 0x7E


def test_fp4_pv_is_attention_and_coarser_than_the_method():
    """Against exact attention on a generated workload the assignment is a (coarse) approximation of the same
    function, with a larger error than NVFP4 + FP8; causal rows see only their keys."""
    w = wl.prefill_workload("t", 23, 1, 384, 4, 2, True)
    qb, kb, vb = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    z = orc.stage1(qb, kb, vb)
    d_v = float(np.float32(np.abs(orc.bits_to_f32(vb)).max() / (6.0 * 448.0)))
    vc, vs = orc.quantize_v_fp4(vb, d_v)
    rows = orc.all_rows(1, 4, 384)
    o4, _ = orc.prefill_rows_pv_fp4(z, vc, vs, d_v, rows, w.softmax_scale, True)
    o8, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    ex = orc.exact_rows(qb, kb, vb, rows, w.softmax_scale, True)
    e4, e8 = np.abs(o4 - ex).mean(), np.abs(o8 - ex).mean()
    assert e8 < e4 < 0.25 * np.abs(ex).mean() + 0.05
    # row 0 of every head sees key 0 only: P = 1 -> code 6 at scale 448, the output is V-hat of key 0
    deq0 = _signed_vals(_unpack(vc)[0, :, :, 0, 0]) * _e4m3_vals(vs[0, :, :, 0]) * d_v      # [Hkv,128]
    for hq in range(4):
        r = hq * 384
        assert np.abs(o4[r] - deq0[hq // 2]).max() <= 1e-6 * max(1.0, np.abs(deq0).max())


def test_inspection_switches_change_nothing_unless_asked():
    """The hooks a GPU test uses to show that a row differs by one rounding decision: asking for the codes leaves the
    output as it is; moving one key's code or one block's scale by a step changes that row, and only in the way
    the decoded values say."""
    z, s, vb = _case()
    d_v = float(np.float32(np.abs(orc.bits_to_f32(vb)).max() / (6.0 * 448.0)))
    vc, vs = orc.quantize_v_fp4(vb, d_v)
    rows = np.array([[0, 0, 0]], np.int32)
    scale = 0.004
    plain, _ = orc.prefill_rows_pv_fp4(z, vc, vs, d_v, rows, scale, False)
    o, _, pc, ps, y, am = orc.prefill_rows_pv_fp4(z, vc, vs, d_v, rows, scale, False, want_codes=True)
    assert np.array_equal(o, plain)
    # the recorded pre-rounding values are the ones the codes were made from
    assert np.array_equal(_e2m1_codes_rne(y[0]), pc[0])
    assert np.array_equal(_e4m3_codes_rne(am[0]), ps[0])
    key = int(np.nonzero((pc[0] > 1) & (pc[0] < 7))[0][0])
    f1, _, pc1, _, _, _ = orc.prefill_rows_pv_fp4(z, vc, vs, d_v, rows, scale, False, want_codes=True, flip_key=key, flip_dir=1)
    assert pc1[0, key] == pc[0, key] + 1 and (np.delete(pc1[0], key) == np.delete(pc[0], key)).all()
    assert np.abs(f1 - plain).max() > 0
    blk = key // 16
    f2, _, pc2, ps2, _, _ = orc.prefill_rows_pv_fp4(z, vc, vs, d_v, rows, scale, False, want_codes=True, flip_blk=blk, flip_blk_dir=-1)
    assert ps2[0, blk] == ps[0, blk] - 1 and (np.delete(ps2[0], blk) == np.delete(ps[0], blk)).all()
    assert np.array_equal(pc2[0, :16 * blk], pc[0, :16 * blk]) and np.array_equal(pc2[0, 16 * blk + 16:], pc[0, 16 * blk + 16:])
    assert np.abs(f2 - plain).max() > 0

"""GPU parity: the prefill kernel against the oracle's emulated QK4PV8 output.

Tolerance (the benchmark spec): max-abs 2e-3 and mean-abs 2e-4 against the oracle.  The kernel's FP32
result before the final rounding is compared under exactly that bound; the BF16 result must be
the round-to-nearest-even image of that FP32 value and, against the oracle, either within
2e-3 or one of the two BF16 neighbours of the oracle's FP32 value (a BF16 ulp above 0.25 is
already larger than 2e-3, so a one-ulp rounding flip cannot be held to the bound)."""
import os

import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-3, 2e-4


def bf16_neighbours_ok(got_bits: np.ndarray, ref32: np.ndarray) -> np.ndarray:
    """True where the BF16 value is within 2e-3 of ref32 or is one of its two BF16 neighbours."""
    got = orc.bits_to_f32(got_bits)
    lo = (ref32.view(np.uint32) & 0xFFFF0000).view(np.float32)              # truncation toward zero
    hi = ((ref32.view(np.uint32) & 0xFFFF0000) + 0x10000).view(np.float32)  # next magnitude up
    return (np.abs(got - ref32) <= MAX_ABS) | (got == lo) | (got == hi)


def compare(o16_gpu, o32_gpu, rows, ref32, label=""):
    g32 = o32_gpu[rows[:, 0], rows[:, 2], rows[:, 1]]
    g16 = o16_gpu[rows[:, 0], rows[:, 2], rows[:, 1]]
    d = np.abs(g32 - ref32)
    assert np.isfinite(g32).all(), label
    assert d.max() <= MAX_ABS, (label, float(d.max()))
    assert d.mean() <= MEAN_ABS, (label, float(d.mean()))
    # BF16 output = RNE of the kernel's FP32 value
    want16 = torch.from_numpy(g32.copy()).to(torch.bfloat16).view(torch.uint16).numpy()
    assert np.array_equal(g16, want16), label
    assert bf16_neighbours_ok(g16, ref32).all(), label
    assert np.abs(orc.bits_to_f32(g16) - ref32).mean() <= MEAN_ABS + 2e-3 * np.abs(ref32).mean(), label
    return float(d.max()), float(d.mean())


def run_gpu(w, smooth=True, use_delta=True, v_scale=1.0):
    from paper_2609_33135_b200 import binding
    s1 = binding.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda(), smooth=smooth, v_scale=v_scale)
    if not use_delta:
        s1.delta = None
    out, o32, status = binding.prefill(s1, w.causal, w.softmax_scale, want_f32=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy()


CASES = {
    "cfg1": lambda: wl.config1_tiny(),
    "cfg1b_qbias": lambda: wl.config1b_tiny_qbias(),
    "causal_128": lambda: wl.prefill_workload("c128", 51, 1, 128, 1, 1, True),
    "causal_384_gqa": lambda: wl.prefill_workload("c384", 52, 1, 384, 4, 2, True, q_bias=True),
    "ragged_causal": lambda: wl.prefill_workload("rag", 53, 2, 333, 4, 2, True, q_bias=True),
    "ragged_noncausal_nq_lt_nkv": lambda: wl.prefill_workload("rag2", 54, 1, 517, 2, 1, False, N_q=200),
    "causal_offset": lambda: wl.prefill_workload("coff", 55, 1, 640, 2, 2, True, N_q=130, q_bias=True),
    # more queries than keys under a bottom-right aligned causal mask: the first 300 rows see no key (output 0),
    # two whole query tiles have no KV block to visit
    "causal_nq_gt_nkv": lambda: wl.prefill_workload("cgt", 56, 1, 200, 2, 1, True, N_q=500, q_bias=True),
    # 320 one-block work items on 148 persistent CTAs: item boundaries back to back
    "many_one_block_items": lambda: wl.prefill_workload("one", 57, 1, 128, 8, 2, False, N_q=5120, q_bias=True),
    # 2- and 3-block items only
    "many_short_items": lambda: wl.prefill_workload("short", 58, 2, 300, 8, 4, False, N_q=1500),
}


@pytest.mark.parametrize("name", list(CASES))
def test_prefill_matches_oracle_all_rows(name):
    w = CASES[name]()
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, w.causal)
    o16, o32 = run_gpu(w)
    compare(o16, o32, rows, ref32, name)


def test_prefill_direct_and_no_compensation_variants():
    w = CASES["causal_384_gqa"]()
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    q, k, v = orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v)
    zd = orc.stage1(q, k, v, smooth=False, v_scale=2.0)
    ref32, _ = orc.prefill_rows(zd, rows, w.softmax_scale, True)
    o16, o32 = run_gpu(w, smooth=False, v_scale=2.0)
    compare(o16, o32, rows, ref32, "direct")
    zs = orc.stage1(q, k, v)
    ref32, _ = orc.prefill_rows(zs, rows, w.softmax_scale, True, use_delta=False)
    o16, o32 = run_gpu(w, use_delta=False)
    compare(o16, o32, rows, ref32, "smoothed, compensation off")
    # and the three differ from one another (the compensation MMA really contributes)
    with_c, _ = orc.prefill_rows(zs, rows, w.softmax_scale, True)
    assert np.abs(with_c - ref32).max() > 1e-2


def test_prefill_bitwise_repeatable():
    w = CASES["ragged_causal"]()
    a16, a32 = run_gpu(w)
    b16, b32 = run_gpu(w)
    assert np.array_equal(a16, b16) and np.array_equal(a32.view(np.uint32), b32.view(np.uint32))


def test_prefill_multi_tile_sampled_rows():
    """Several hundred CTAs, 32 KV blocks per row at the end: parity on a stratified row sample."""
    w = wl.prefill_workload("mid", 56, 1, 4096, 8, 2, True, q_bias=True)
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = wl.sample_rows(56, w.B, w.H_q, w.N_q, 256).numpy()
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    o16, o32 = run_gpu(w)
    compare(o16, o32, rows, ref32, "4k")


def test_prefill_elementwise_compensation_variant():
    """Ablation variant (Section 7.4): Delta_S added by the softmax threads instead of the seed MMA.  Checked against
    the oracle's statement of that placement; against the product path the outputs may differ by the place of one
    FP32 rounding per score (on small inputs they are often identical)."""
    from paper_2609_33135_b200 import binding as B_
    w = wl.prefill_workload("ew", 59, 2, 333, 4, 2, True, q_bias=True)
    s1 = B_.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda())
    out = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.bfloat16, device="cuda")
    o32 = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_variant(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, 1.0, True, w.softmax_scale,
                            B_.MPFA_VARIANT_COMP_ELEMENTWISE, out, o32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True, elementwise=True)
    compare(out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy(), rows, ref32, "elementwise")
    _, seeded32, _ = B_.prefill(s1, True, w.softmax_scale, want_f32=True)
    torch.cuda.synchronize()
    d = (seeded32 - o32).abs()
    assert float(d.mean()) < 1e-4
    # variant 0 is the product path itself
    o32b = torch.empty_like(o32)
    B_.mpfa_prefill_variant(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, 1.0, True, w.softmax_scale, 0, out, o32b, status)
    torch.cuda.synchronize()
    assert torch.equal(o32b, seeded32)
    with pytest.raises(Exception):
        B_.mpfa_prefill_variant(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, 1.0, True, w.softmax_scale, 7, out, o32b, status)


@pytest.mark.parametrize("kind", ["zeros", "zero_blocks", "constant"])
def test_prefill_on_degenerate_inputs(kind):
    """All-zero tensors (tensor scale 1, every score 0: the output is the plain mean of the visible V rows), zero
    blocks and heads, and sequences whose tokens are all identical (centered values exactly zero, the scores come
    from the compensation term alone)."""
    from test_gpu_quantize import _adversarial
    w = _adversarial(kind, 500 + len(kind))
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    o16, o32 = run_gpu(w)
    # Both sides decide the E4M3 code of P-hat in FP32 from 448 P; the one input of that decision they do not share
    # bit for bit is 2^x (hardware approximation within 2 ulp on the GPU, correctly rounded in the oracle).  A row may
    # therefore exceed the bound only if that is demonstrably what happened: the oracle's own 448 P of one of its
    # keys lies within 2e-6 (relative) of an E4M3 rounding boundary, and the oracle with exactly that key's code moved
    # one step across that boundary reproduces the kernel's row within the usual bound.  On structured workloads no
    # row needs this; on these structureless N(0,1) tensors one row in a few thousand does (few dozen keys, so one
    # 6 % step of one P moves the output by a few 1e-3).
    g32 = o32[rows[:, 0], rows[:, 2], rows[:, 1]]
    d = np.abs(g32 - ref32)
    assert np.isfinite(g32).all()
    assert d.mean() <= MEAN_ABS, (kind, float(d.mean()))
    over = np.nonzero(d.max(axis=1) > MAX_ABS)[0]
    assert len(over) <= max(1, len(rows) // 1000), (kind, len(over))
    grid = np.array([orc.e4m3_decode(c) for c in range(0x7F)], np.float64)
    bounds = (grid[1:] + grid[:-1]) / 2                      # rounding boundaries between adjacent codes
    for r in over:
        row = rows[r:r + 1]
        codes, _, q, _ = orc.phat_rows(z, row, w.softmax_scale, True, want_q=True)
        n_vis = int(row[0, 2]) + 1 + (w.N_kv - w.N_q)
        qv = q[0, :n_vis].astype(np.float64)
        nearest = np.abs(qv[:, None] - bounds[None, :])
        j = nearest.argmin(axis=1)
        rel = nearest[np.arange(n_vis), j] / np.maximum(bounds[j], 1e-30)
        cands = np.nonzero(rel <= 2e-6)[0]
        assert len(cands) >= 1, (kind, row, float(d[r].max()), float(rel.min()))
        explained = False
        for key in cands:
            direction = 1 if codes[0, key] == j[key] else -1   # code below the boundary moves up, and the reverse
            _, _, _, o_flip = orc.phat_rows(z, row, w.softmax_scale, True, want_q=True, flip_key=int(key), flip_dir=direction)
            if np.abs(g32[r] - o_flip[0]).max() <= MAX_ABS:
                explained = True
                print(f"{kind}: row {row[0].tolist()} differs by {d[r].max():.2e}: key {key} has 448 P = {qv[key]:.9g}, "
                      f"{rel[key]:.1e} from the boundary {bounds[j[key]]:.9g} between codes {j[key]:#x} and {j[key] + 1:#x}; "
                      f"with that code moved one step the oracle is within {np.abs(g32[r] - o_flip[0]).max():.1e}")
                break
        assert explained, (kind, row, float(d[r].max()))
    keep = d.max(axis=1) <= MAX_ABS
    compare(o16, o32, rows[keep], ref32[keep], kind)

def test_prefill_many_items_without_keys_per_cta():
    """Causal, far more queries than keys (N_q = 8192, N_kv = 128, 32 heads): 63 of the 64 query tiles see no key at
    all, so every persistent CTA walks a dozen and more empty work items in a row.  They must come out as zeros,
    the live tile must match the oracle, and no bounded wait may run out (status 0)."""
    w = wl.prefill_workload("empty_items", 61, 1, 128, 32, 8, True, N_q=8192, q_bias=True)
    from paper_2609_33135_b200 import binding
    s1 = binding.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda())
    for _ in range(2):
        out, o32, status = binding.prefill(s1, True, w.softmax_scale, want_f32=True)
        out.fill_(3.0)
        o32.fill_(3.0)
        status.zero_()
        binding.mpfa_prefill(s1.q, s1.k, s1.v_fp8, s1.delta, s1.stats, 1.0, True, w.softmax_scale, out, o32, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        o16n, o32n = out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy()
        assert not o32n[0, :8192 - 128].any() and not o16n[0, :8192 - 128].any()
        z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
        rows = orc.all_rows(1, 32, 8192)
        rows = rows[rows[:, 2] >= 8192 - 128]
        ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
        compare(o16n, o32n, rows, ref32, "empty items")


@pytest.fixture
def two_tile_arrangement():
    from paper_2609_33135_b200 import binding
    binding.mpfa_set_prefill_arrangement(1)
    yield
    binding.mpfa_set_prefill_arrangement(int(os.environ.get("MPFA_TEST_ARRANGEMENT", "0")))   # what the suite runs on


@pytest.mark.parametrize("name", ["cfg1b_qbias", "causal_384_gqa", "ragged_causal", "ragged_noncausal_nq_lt_nkv",
                                  "causal_offset", "causal_nq_gt_nkv", "many_one_block_items", "many_short_items"])
def test_two_tile_arrangement_matches_oracle(two_tile_arrangement, name):
    """Section 5.1's arrangement (two query tiles per CTA, a softmax warpgroup and an accumulator each) is the same
    arithmetic row by row: same oracle, same tolerance.  Odd tile counts leave one stage of the last pair idle."""
    w = CASES[name]()
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, w.causal)
    o16, o32 = run_gpu(w)
    compare(o16, o32, rows, ref32, name)


def test_two_tile_arrangement_sampled_rows_and_empty_items(two_tile_arrangement):
    w = wl.prefill_workload("mid2", 62, 1, 4096 + 128, 8, 2, True, q_bias=True)   # odd number of query tiles
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = wl.sample_rows(62, w.B, w.H_q, w.N_q, 256).numpy()
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    o16, o32 = run_gpu(w)
    compare(o16, o32, rows, ref32, "4k+128, two tiles per CTA")
    test_prefill_many_items_without_keys_per_cta()


@pytest.mark.parametrize("name", ["cfg1b_qbias", "causal_384_gqa", "ragged_causal", "ragged_noncausal_nq_lt_nkv",
                                  "causal_offset", "many_short_items"])
def test_prefill_bf16_pv_variant_matches_its_oracle(name):
    """Section 3.1's NVFP4 + BF16 precision assignment (mpfa_prefill_variant, MPFA_VARIANT_PV_BF16): the same logits,
    P in BF16, V unquantized.  Held to the same tolerance against the oracle's statement of that assignment; a BF16
    rounding of P is a 2^-9 step, and 2^x within 2 ulp cannot move it except on a boundary, as for the FP8 codes."""
    from paper_2609_33135_b200 import binding as B_
    w = CASES[name]()
    s1 = B_.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda())
    vt = B_.mpfa_pack_v_bf16(w.v.cuda())
    out = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.bfloat16, device="cuda")
    o32 = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_variant(s1.q, s1.k, vt, s1.delta, s1.stats, 1.0, w.causal, w.softmax_scale, B_.MPFA_VARIANT_PV_BF16,
                            out, o32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(w.B, w.H_q, w.N_q)
    ref32, _ = orc.prefill_rows_pv_bf16(z, orc.bf16_bits(w.v), rows, w.softmax_scale, w.causal)
    compare(out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy(), rows, ref32, name + " (BF16 P V)")
    # and it is a different function from the product path
    m32, _ = orc.prefill_rows(z, rows, w.softmax_scale, w.causal)
    assert np.abs(m32 - ref32).mean() > 1e-4


def test_prefill_bf16_pv_variant_sampled_rows_4k():
    from paper_2609_33135_b200 import binding as B_
    w = wl.prefill_workload("mid3", 63, 1, 4096, 8, 2, True, q_bias=True)
    s1 = B_.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda())
    vt = B_.mpfa_pack_v_bf16(w.v.cuda())
    out = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.bfloat16, device="cuda")
    o32 = torch.empty(w.B, w.N_q, w.H_q, 128, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B_.mpfa_prefill_variant(s1.q, s1.k, vt, s1.delta, s1.stats, 1.0, True, w.softmax_scale, B_.MPFA_VARIANT_PV_BF16, out, o32,
                            status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = wl.sample_rows(63, w.B, w.H_q, w.N_q, 256).numpy()
    ref32, _ = orc.prefill_rows_pv_bf16(z, orc.bf16_bits(w.v), rows, w.softmax_scale, True)
    compare(out.view(torch.uint16).cpu().numpy(), o32.cpu().numpy(), rows, ref32, "4k (BF16 P V)")

"""GPU parity: stage-1 kernels against the oracle, bit for bit (codes, block scales, tensor
scales, means, compensation vector, V codes), through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

from layouts import codes_to_logical, pad128, sf_to_logical

pytestmark = pytest.mark.gpu


def _cases():
    return {
        "cfg1": lambda: wl.config1_tiny(),
        "cfg1b": lambda: wl.config1b_tiny_qbias(),
        "ragged_gqa": lambda: wl.prefill_workload("ragged", 41, 2, 333, 4, 2, True, N_q=300, q_bias=True),
        "gqa5_2k": lambda: wl.prefill_workload("gqa5", 42, 1, 2048 + 77, 10, 2, True, q_bias=True),
    }


def run_stage1_gpu(w, smooth=True, v_scale=1.0):
    from paper_2609_33135_b200 import binding
    return binding.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda(), smooth=smooth, v_scale=v_scale)


def check_stage1(w, s1, z, smooth=True):
    B, Nq, Hq, Nkv, Hkv = w.B, w.N_q, w.H_q, w.N_kv, w.H_kv
    torch.cuda.synchronize()
    assert np.array_equal(s1.stats.q_mean.cpu().numpy(), z.q_mean)
    assert np.array_equal(s1.stats.k_mean.cpu().numpy(), z.k_mean)
    assert np.array_equal(s1.stats.q_gscale.cpu().numpy(), z.dq)
    assert np.array_equal(s1.stats.k_gscale.cpu().numpy(), z.dk)
    for t, codes, sf, H, N in ((s1.q, z.q_codes, z.q_sf, Hq, Nq), (s1.k, z.k_codes, z.k_sf, Hkv, Nkv)):
        got, padrows = codes_to_logical(t.codes.cpu().numpy(), B, H, N)
        assert np.array_equal(got, codes)
        assert not padrows.any()
        gsf = sf_to_logical(t.sf.cpu().numpy(), B, H, N)
        assert np.array_equal(gsf[:, :, :N], sf)
        assert not gsf[:, :, N:].any()
    gv = s1.v_fp8.cpu().numpy().reshape(B, Hkv, pad128(Nkv), 128)
    assert np.array_equal(gv[:, :, :Nkv], z.v_codes)
    assert not gv[:, :, Nkv:].any()
    if smooth:
        gd = s1.delta.view(torch.uint16).cpu().numpy()
        assert np.array_equal(gd[:, :, :Nkv], z.delta)
        assert not gd[:, :, Nkv:].any()
    else:
        assert s1.delta is None


@pytest.mark.parametrize("name", list(_cases()))
def test_stage1_bit_exact(name):
    w = _cases()[name]()
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    check_stage1(w, run_stage1_gpu(w), z)


def test_stage1_direct_variant_and_v_scale():
    w = _cases()["ragged_gqa"]()
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v), smooth=False, v_scale=0.5)
    s1 = run_stage1_gpu(w, smooth=False, v_scale=0.5)
    check_stage1(w, s1, z, smooth=False)
    assert not s1.stats.q_mean.any() and not s1.stats.k_mean.any()


def test_frozen_statistics_single_token_query():
    """Decode-time query: one token centered and scaled with the frozen prefill statistics."""
    from paper_2609_33135_b200 import binding
    w = _cases()["ragged_gqa"]()
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    s1 = run_stage1_gpu(w)
    qn = w.q[:, 17:18].contiguous()
    zq = orc.stage1(orc.bf16_bits(qn), orc.bf16_bits(w.k), orc.bf16_bits(w.v), frozen=z)
    q4 = binding.Fp4Tensor.empty(w.B, w.H_q, 1)
    binding.mpfa_quantize_qk(qn.cuda(), None, binding.MPFA_SMOOTH | binding.MPFA_STATS_FROZEN, s1.stats, q4, None,
                             None, None)
    torch.cuda.synchronize()
    got, pad = codes_to_logical(q4.codes.cpu().numpy(), w.B, w.H_q, 1)
    assert np.array_equal(got, zq.q_codes) and not pad.any()
    assert np.array_equal(sf_to_logical(q4.sf.cpu().numpy(), w.B, w.H_q, 1)[:, :, :1], zq.q_sf)


def test_deterministic_and_argument_errors():
    from paper_2609_33135_b200 import binding
    w = _cases()["cfg1b"]()
    a = run_stage1_gpu(w)
    b = run_stage1_gpu(w)
    torch.cuda.synchronize()
    assert torch.equal(a.q.codes, b.q.codes) and torch.equal(a.k.sf, b.k.sf) and torch.equal(a.delta, b.delta)
    q = w.q.cuda()
    st = binding.Stats.empty(1, 1, 1)
    q4 = binding.Fp4Tensor.empty(1, 1, 256)
    ws = binding.quantize_workspace(1, 1, 1)
    with pytest.raises(binding.MpfaError, match="workspace"):
        binding.mpfa_quantize_qk(q, None, 0, st, q4, None, None, ws[:256])
    with pytest.raises(binding.MpfaError, match="misaligned"):
        bad = binding.Fp4Tensor(q4.codes[16:], q4.sf, 1, 1, 255)
        binding.mpfa_quantize_qk(q[:, :255].contiguous(), None, 0, st, bad, None, None, ws)
    with pytest.raises(binding.MpfaError, match="invalid"):
        binding.mpfa_quantize_qk(q, None, 0, st, binding.Fp4Tensor(q4.codes, q4.sf, 1, 1, 128), None, None, ws)


def _adversarial(kind: str, seed: int):
    """Small tensors with the values that break sloppy quantizers: hand-built, not drawn from the workload recipe."""
    import dataclasses
    g = torch.Generator().manual_seed(seed)
    B, N, Hq, Hkv = 2, 300, 4, 2
    q = torch.randn(B, N, Hq, 128, generator=g)
    k = torch.randn(B, N, Hkv, 128, generator=g)
    v = torch.randn(B, N, Hkv, 128, generator=g)
    if kind == "zeros":                 # an all-zero batch element (tensor scale 1) next to an ordinary one
        q[0].zero_(); k[0].zero_(); v[0].zero_()
    elif kind == "zero_blocks":         # blocks and whole heads of zeros inside a non-zero tensor, negative zeros
        k[:, :, 0, :].zero_(); q[:, :, 1, 32:48] = 0.0; q[:, ::2, 2, :] = -0.0; v[:, 5:9] = -0.0
    elif kind == "dynamic_range":       # 2^-120 .. 2^100 in one tensor: scales underflow to 0 and saturate at 448
        e = torch.randint(-120, 100, (B, N, Hkv, 128), generator=g).float()
        k = k.sign() * torch.exp2(e)
        q = q * 1e-30
        v = v * 1e30
    elif kind == "ties":                # values on the E2M1 and E4M3 rounding boundaries after scaling
        grid = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 0.0, 7.0])
        idx = torch.randint(0, 16, (B, N, Hkv, 128), generator=g)
        k = grid[idx] * k.sign()
        k[:, 0, :, 0] = 6.0 * 448.0 / 448.0
        q = (torch.randint(-8, 9, (B, N, Hq, 128), generator=g).float()) * 0.25
        v = torch.randint(-32, 33, (B, N, Hkv, 128), generator=g).float() * 0.0625 + 448.0 * (torch.rand(B, N, Hkv, 128, generator=g) < 0.01)
    elif kind == "constant":            # every token identical: centered values are exactly zero
        q = q[:, :1].expand(B, N, Hq, 128).clone(); k = k[:, :1].expand(B, N, Hkv, 128).clone()
    w = wl.prefill_workload("adv", 1, B, N, Hq, Hkv, True)
    return dataclasses.replace(w, q=q.to(torch.bfloat16), k=k.to(torch.bfloat16), v=v.to(torch.bfloat16))


@pytest.mark.parametrize("kind", ["zeros", "zero_blocks", "dynamic_range", "ties", "constant"])
def test_stage1_bit_exact_on_adversarial_values(kind):
    w = _adversarial(kind, 400 + len(kind))
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    check_stage1(w, run_stage1_gpu(w), z)


def test_means_are_deterministic_on_unflushed_inputs():
    """Eq. 7 on inputs the seeded generator never produces: magnitudes from 2^-60 up to O(1) mixed in every column,
    so the FP64 column sums are no longer exact and their value depends on the order of addition.  The kernels add
    in a fixed order (no floating-point atomics): two runs must agree bit for bit in every output, and the means
    must be within one FP32 ulp of the oracle's single ascending sum."""
    from paper_2609_33135_b200 import binding
    g = torch.Generator(device="cpu").manual_seed(77)
    B, N, Hq, Hkv = 2, 3000, 4, 2
    def draw(H):
        x = torch.randn(B, N, H, 128, generator=g)
        e = torch.randint(-60, 1, (B, N, H, 128), generator=g).float()
        return (x * torch.exp2(e)).to(torch.bfloat16)
    q, k, v = draw(Hq), draw(Hkv), draw(Hkv)
    assert float(q.float().abs()[q.float().abs() > 0].min()) < 2.0 ** -55
    runs = []
    for _ in range(2):
        s1 = binding.stage1(q.cuda(), k.cuda(), v.cuda())
        torch.cuda.synchronize()
        runs.append([t.clone() for t in (s1.stats.q_mean, s1.stats.k_mean, s1.stats.q_gscale, s1.stats.k_gscale, s1.q.codes,
                                         s1.q.sf, s1.k.codes, s1.k.sf, s1.delta.view(torch.uint16))])
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    for got, x in ((runs[0][0], q), (runs[0][1], k)):
        ref = orc.means(orc.bf16_bits(x))
        got = got.cpu().numpy()
        ulp = np.spacing(np.abs(ref).astype(np.float32))
        assert np.all(np.abs(got.astype(np.float64) - ref.astype(np.float64)) <= ulp)
        assert (got == ref).mean() > 0.99


def test_stage1_with_a_one_slice_workspace_is_the_same_on_exact_inputs():
    """The statistics pass takes as many token slices as the workspace holds; on the generator's inputs (exact
    sums) the slice count cannot change a bit."""
    from paper_2609_33135_b200 import binding
    w = wl.prefill_workload("ws", 43, 1, 2500, 4, 2, True, q_bias=True)
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    n_min = binding.lib().mpfa_quantize_workspace_min_bytes(1, 4, 2)
    assert n_min < binding.lib().mpfa_quantize_workspace_bytes(1, 4, 2)
    for nbytes in (n_min, 3 * n_min):
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        check_stage1(w, binding.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda(), workspace=ws), z)
    with pytest.raises(binding.MpfaError, match="workspace"):
        binding.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda(), workspace=torch.empty(n_min - 256, dtype=torch.uint8, device="cuda"))

"""The workspace-free stage-1 entry point (mpfa_quantize_qk_static) against the regular one.

Some embedders can pass the library nothing but inputs and outputs: no scratch pointer and
no way to allocate one.  For them the library carries a fixed scratch buffer of its own.  This
test calls that entry point through the C ABI twice in a row, on two different inputs, and
requires bit-identical outputs to mpfa_quantize_qk (the quantizers are specified to the bit),
which also shows that the second call is not disturbed by what the first left in the shared
buffer.  It runs last so that a failure here cannot hide the other tests' results."""
import pytest
import torch

from paper_2609_33135_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _both(binding, w):
    B, Nq, Hq, Nkv, Hkv = w.B, w.N_q, w.H_q, w.N_kv, w.H_kv
    q, k = w.q.cuda(), w.k.cuda()
    outs = []
    for static in (False, True):
        st = binding.Stats.empty(B, Hq, Hkv)
        q4, k4 = binding.Fp4Tensor.empty(B, Hq, Nq), binding.Fp4Tensor.empty(B, Hkv, Nkv)
        delta = torch.zeros(B, Hq, (Nkv + 127) // 128 * 128, dtype=torch.bfloat16, device="cuda")
        if static:
            binding.mpfa_quantize_qk_static(q, k, binding.MPFA_SMOOTH, st, q4, k4, delta)
        else:
            ws = binding.quantize_workspace(B, Hq, Hkv)
            binding.mpfa_quantize_qk(q, k, binding.MPFA_SMOOTH, st, q4, k4, delta, ws)
        torch.cuda.synchronize()
        outs.append((st, q4, k4, delta))
    return outs


def _assert_same(a, b):
    (sa, qa, ka, da), (sb, qb, kb, db) = a, b
    assert torch.equal(sa.q_mean, sb.q_mean) and torch.equal(sa.k_mean, sb.k_mean)
    assert torch.equal(sa.q_gscale, sb.q_gscale) and torch.equal(sa.k_gscale, sb.k_gscale)
    assert torch.equal(qa.codes, qb.codes) and torch.equal(qa.sf, qb.sf)
    assert torch.equal(ka.codes, kb.codes) and torch.equal(ka.sf, kb.sf)
    assert torch.equal(da.view(torch.uint16), db.view(torch.uint16))
    assert sa.q_mean.abs().max() > 0 and ka.codes.any()


def test_static_scratch_entry_point_matches_twice_in_a_row():
    from paper_2609_33135_b200 import binding
    first = wl.prefill_workload("na1", 91, 2, 333, 8, 2, True, N_q=300, q_bias=True)
    second = wl.prefill_workload("na2", 92, 1, 1000, 4, 4, False, q_bias=True)
    for w in (first, second):      # back to back: the second call reuses the same device buffer
        regular, static = _both(binding, w)
        _assert_same(regular, static)


def test_static_scratch_rejects_oversized_shapes():
    from paper_2609_33135_b200 import binding
    limit = binding.lib().mpfa_static_scratch_bytes()
    B, Hq, Hkv = 16, 40, 8
    assert binding.lib().mpfa_quantize_workspace_min_bytes(B, Hq, Hkv) > limit
    q = torch.zeros(B, 4, Hq, 128, dtype=torch.bfloat16, device="cuda")
    st = binding.Stats.empty(B, Hq, Hkv)
    q4 = binding.Fp4Tensor.empty(B, Hq, 4)
    with pytest.raises(binding.MpfaError, match="workspace too small"):
        binding.mpfa_quantize_qk_static(q, None, 0, st, q4, None, None)


def test_static_scratch_frozen_statistics_have_no_size_limit_and_nothing_is_allocated():
    """With frozen statistics the quantizer accumulates nothing, so the fixed buffer is not used and the size limit
    does not apply: the decode-time query batch of the paged-decode configuration (32 requests, 32 + 8 heads) goes
    through although its statistics would not fit.  Also checks what the entry point is for: across the call the
    device allocator's books and the driver's free-memory figure do not move."""
    from paper_2609_33135_b200 import binding
    B, Hq, Hkv = 32, 32, 8
    assert binding.lib().mpfa_quantize_workspace_min_bytes(B, Hq, Hkv) > binding.lib().mpfa_static_scratch_bytes()
    g = torch.Generator(device="cpu").manual_seed(5)
    q = torch.randn(B, 1, Hq, 128, generator=g).to(torch.bfloat16).cuda()
    st = binding.Stats.empty(B, Hq, Hkv)
    st.q_mean.copy_(torch.randn(B, Hq, 128, generator=g) * 0.1)
    st.q_gscale.fill_(0.002)
    st.k_gscale.fill_(0.01)
    flags = binding.MPFA_SMOOTH | binding.MPFA_STATS_FROZEN
    ref = binding.Fp4Tensor.empty(B, Hq, 1)
    binding.mpfa_quantize_qk(q, None, flags, st, ref, None, None, None)
    out = binding.Fp4Tensor.empty(B, Hq, 1)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(2):
        binding.mpfa_quantize_qk_static(q, None, flags, st, out, None, None)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert free1 == free0
    assert torch.equal(out.codes, ref.codes) and torch.equal(out.sf, ref.sf)
    assert out.codes.any()

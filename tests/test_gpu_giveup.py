"""The bounded device waits, exercised the safe way: a test-only build of the library whose waits give up after a
few milliseconds and whose CTA 0 leaves out one shared-memory copy, so that one wait really runs out.  Nothing
faults or spins without bound: the kernel raises MPFA_DEV_TIMEOUT in *device_status, every role leaves its loops,
copies still in flight are awaited, tensor memory is released and the call returns.  The product library, used
right afterwards in the same process, must be unaffected."""
import time

import numpy as np
import pytest
import torch

from oracle import mpfa_oracle as orc
from paper_2609_33135_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def giveup_lib():
    from paper_2609_33135_b200 import binding, build
    return binding.load_library(build.build_giveup_test_lib())


@pytest.fixture
def use_giveup_lib(giveup_lib):
    from paper_2609_33135_b200 import binding
    product = binding.lib()
    binding._lib = giveup_lib
    yield
    binding._lib = product
    binding.mpfa_set_prefill_arrangement(0)


def _prefill_case():
    w = wl.prefill_workload("giveup", 81, 1, 640, 4, 2, True, q_bias=True)
    z = orc.stage1(orc.bf16_bits(w.q), orc.bf16_bits(w.k), orc.bf16_bits(w.v))
    rows = orc.all_rows(1, 4, 640)
    ref32, _ = orc.prefill_rows(z, rows, w.softmax_scale, True)
    return w, rows, ref32


@pytest.mark.parametrize("arrangement", [0, 1])
def test_prefill_wait_runs_out_and_the_call_returns(use_giveup_lib, giveup_lib, arrangement):
    from paper_2609_33135_b200 import binding
    w, rows, ref32 = _prefill_case()
    giveup_lib.mpfa_set_prefill_arrangement(arrangement)
    s1 = binding.stage1(w.q.cuda(), w.k.cuda(), w.v.cuda())      # stage 1 has no waits: unaffected
    torch.cuda.synchronize()
    t0 = time.time()
    out, o32, status = binding.prefill(s1, True, w.softmax_scale, want_f32=True)
    torch.cuda.synchronize()
    assert time.time() - t0 < 5.0
    assert int(status.item()) & binding.MPFA_DEV_TIMEOUT
    # the same process, the product library, right afterwards: correct result, clean status
    binding._lib = binding.load_library(binding.LIB_PATH)
    binding.mpfa_set_prefill_arrangement(arrangement)
    out, o32, status = binding.prefill(s1, True, w.softmax_scale, want_f32=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = o32.cpu().numpy()[rows[:, 0], rows[:, 2], rows[:, 1]]
    err = np.abs(got - ref32)
    assert err.max() <= 2e-3 and err.mean() <= 2e-4
    binding.mpfa_set_prefill_arrangement(0)


def test_decode_wait_runs_out_and_the_call_returns(use_giveup_lib):
    from paper_2609_33135_b200 import binding, decode_cache
    dw = wl.decode_workload("giveup_decode", 82, 2, 8, 2, 64, 1500, seq_lens=[1500, 700])
    st = decode_cache.build_cache(dw)            # cache writes have no waits
    torch.cuda.synchronize()
    t0 = time.time()
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert time.time() - t0 < 5.0
    assert int(st.status.item()) & binding.MPFA_DEV_TIMEOUT
    binding._lib = binding.load_library(binding.LIB_PATH)
    st.status.zero_()
    decode_cache.decode_step(st)
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0
    for b in range(dw.B):
        k, v = dw.kv_for_request(b)
        zc = orc.stage1(orc.bf16_bits(dw.q_sample[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v))
        zq = orc.stage1(orc.bf16_bits(dw.q_new[b:b + 1].contiguous()), orc.bf16_bits(k), orc.bf16_bits(v), frozen=zc)
        ref, _ = orc.decode(zq.q_codes[:, :, 0], zq.q_sf[:, :, 0], zc.k_codes, zc.k_sf, zc.v_codes, zc.delta, zc.dq,
                            zc.dk, 1.0, dw.softmax_scale, np.array([int(dw.seq_lens[b])], np.int32))
        e = np.abs(st.out_f32[b].cpu().numpy() - ref[0])
        assert e.max() <= 2e-3 and e.mean() <= 2e-4

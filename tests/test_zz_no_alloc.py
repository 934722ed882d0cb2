"""The allocation-free product entry point, checked against the ordinary one.

qift_w2a4_linear_static exists for callers that cannot obtain device memory when they need the
layer (no allocator handed to them, allocation forbidden or synchronizing in their region, a pool
owned by someone else): its int8 scratch is an array compiled into the library.  It must give
exactly what qift_w2a4_linear gives with a caller-provided workspace -- same INT32 accumulators,
same outputs -- and keep doing so when called again, since every call reuses the one array and
inherits the previous call's bytes.  This file sorts last so that a run stopping at the first
failure has already executed every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def problem(lv, M, N, K, seed):
    W = synth.gaussian_weights(seed, N, K)
    x, _ = synth.activations(seed + 1, M, K, max(1, K // 100))
    packed, s_n = qift.qift_pack_weights(dev(W), lv, qift.SCALE_ABSMAX)
    q_a, s_a = qift.qift_quantize_act(dev(x), synth.had_block_for(K), 0.9)
    return packed, s_n, q_a, s_a


def test_static_scratch_matches_the_workspace_entry_point_twice_in_a_row():
    assert qift.qift_static_scratch_bytes() == 16 << 20
    # two different problems back to back: the second inherits the first one's scratch contents,
    # and is smaller, so stale bytes lie right behind the region it rewrites
    cases = [(qift.MNZ, 200, 520, 1024, 11, torch.bfloat16), (qift.POT, 64, 136, 512, 12, torch.float32)]
    for rounds in range(2):
        for lv, M, N, K, seed, dt in cases:
            packed, s_n, q_a, s_a = problem(lv, M, N, K, seed)
            want, want_acc = qift.qift_w2a4_linear(packed, s_n, lv, q_a, s_a, out_dtype=dt, want_acc=True)
            out = torch.empty((M, N), dtype=dt, device="cuda")
            acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
            torch.cuda.synchronize()
            free_before, _ = torch.cuda.mem_get_info()
            got = qift.qift_w2a4_linear_static(packed, s_n, lv, q_a, s_a, out, acc)
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            if rounds > 0:      # past the first call on this device, which loads the kernels
                assert free_after >= free_before, (free_before, free_after)   # no device memory was taken
            assert torch.equal(acc, want_acc)                    # integers: bit for bit
            assert torch.equal(got.view(torch.int16) if dt == torch.bfloat16 else got,
                               want.view(torch.int16) if dt == torch.bfloat16 else want)
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, (rc, detail)


def test_static_scratch_also_agrees_with_the_oracle_and_rejects_oversize():
    lv, M, N, K = qift.SYM, 40, 96, 256
    W = synth.gaussian_weights(5, N, K)
    x, _ = synth.activations(6, M, K, 3)
    p_ref, s_ref, codes = oracle.pack_weights(W, oracle.SYM, oracle.SCALE_ABSMAX)
    q_ref, sa_ref = oracle.quantize_act(x, 256, 0.9)
    y_ref, acc_ref = oracle.linear(codes, oracle.SYM, s_ref, q_ref, sa_ref)
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    qift.qift_w2a4_linear_static(dev(p_ref.view(np.int32)), dev(s_ref), lv, dev(q_ref), dev(sa_ref), out, acc)
    assert np.array_equal(acc.cpu().numpy(), acc_ref) and np.array_equal(out.cpu().numpy(), y_ref)
    # one byte over the capacity is refused on the host, before anything is launched
    big_n, big_k = 4097, 4096
    s_n = torch.ones(big_n, device="cuda")
    q_a = torch.zeros((1, big_k), dtype=torch.int8, device="cuda")
    s_a = torch.ones(4, device="cuda")[:1]
    y = torch.empty((1, big_n), device="cuda")
    packed = torch.zeros(16, dtype=torch.int32, device="cuda")     # never read: the call fails first
    with pytest.raises(qift.QiftError) as e:
        qift.qift_w2a4_linear_static(packed, s_n, lv, q_a, s_a, y)
    assert e.value.status == qift.ERR_TOO_LARGE

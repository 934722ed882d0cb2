"""A bounded device-side wait that really runs out, and what the host sees of it.

Every mbarrier wait in the library gives up after a wall-time bound, records its site in the device
status word and lets the kernel end normally.  qift_selftest_wait_timeout makes that happen on purpose
with a short bound (an mbarrier nobody arrives at; the CTA-pair prefill GEMM starved of its loads) --
no fault, no trap, no unbounded spin -- and these tests follow the report to the host:
QIFT_ERR_TIMEOUT with the site byte, then QIFT_OK, then an ordinary product that still matches the oracle."""
import time

import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def product_still_matches_oracle(M):
    N, K, lv = 272, 512, qift.MNZ
    W = synth.gaussian_weights(77, N, K)
    x, _ = synth.activations(78, M, K, 5)
    p_ref, s_ref, codes = oracle.pack_weights(W, oracle.MNZ, oracle.SCALE_ABSMAX)
    q_ref, sa_ref = oracle.quantize_act(x, 512, 0.9)
    y_ref, acc_ref = oracle.linear(codes, oracle.MNZ, s_ref, q_ref, sa_ref)
    route = qift.ROUTE_PREFILL_PAIR if M > 16 else qift.ROUTE_AUTO
    y, acc = qift.qift_linear_route(dev(p_ref.view(np.int32)), dev(s_ref), lv, dev(q_ref), dev(sa_ref), route, want_acc=True)
    assert np.array_equal(acc.cpu().numpy(), acc_ref) and np.array_equal(y.cpu().numpy(), y_ref)


@pytest.mark.parametrize("which,sites", [(0, {0x7e}), (1, {32, 33})])
def test_expired_wait_is_reported_once_and_the_context_stays_usable(which, sites):
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, (rc, detail)                      # nothing pending from earlier tests
    product_still_matches_oracle(300)                       # loads the kernels, so the timing below is the wait's
    t0 = time.perf_counter()
    qift.qift_selftest_wait_timeout(which, 1000)            # 1 ms bound
    rc, detail = qift.qift_device_status()                  # synchronizes: the kernel has returned by itself
    dt = time.perf_counter() - t0
    assert rc == qift.ERR_TIMEOUT
    assert detail & 0x80000000 and (detail & 0xff) in sites, hex(detail)
    assert dt < 1.0, f"a 1 ms bound took {dt:.3f} s"
    rc, detail = qift.qift_device_status()                  # read-and-clear: the second read is clean
    assert rc == qift.OK and detail == 0
    product_still_matches_oracle(300)                       # same kernel, fed normally: exact again
    product_still_matches_oracle(1)
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, (rc, detail)


def test_selftest_rejects_bad_arguments():
    with pytest.raises(qift.QiftError) as e:
        qift.qift_selftest_wait_timeout(2, 1000)
    assert e.value.status == qift.ERR_INVALID_ARG
    with pytest.raises(qift.QiftError) as e:
        qift.qift_selftest_wait_timeout(0, 0)
    assert e.value.status == qift.ERR_INVALID_ARG
    with pytest.raises(qift.QiftError) as e:
        qift.qift_selftest_wait_timeout(0, 2_000_000)
    assert e.value.status == qift.ERR_INVALID_ARG

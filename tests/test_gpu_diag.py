"""Quantizer diagnostics on the GPU against the oracle: float-grid codes and bucket counts bit-exactly, scales
bit-exactly wherever the sweep's winner is unique, fp64 sums within the tolerance derived below."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift
from conftest import read_golden

pytestmark = pytest.mark.gpu
# Both sides form every squared error from the same fp64 operations; only the ORDER of the fp64 additions differs
# (sequential in the oracle, tree and atomics on the GPU).  Summing n non-negative terms in any order is within
# n * 2^-53 relative of the exact sum; n <= 2^28 here, so 1e-9 relative covers both sides with a wide margin.
SUM_RTOL = 1e-9
# NMSE = f / S2 with f = S2 - 2 beta lin + beta^2 quad: every term is O(S2) and carries the relative error above, so
# the quotient is off by a few 1e-9 ABSOLUTE (not relative: f may cancel to zero).
NMSE_ATOL = 1e-8


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def paper_grids():
    return {r[0]: np.array([float(v) for v in r[1:]], dtype=np.float32)
            for r in read_golden("level_sets.txt") if r[0] != "RATIO"}


def check_scales(W, grid, s_gpu, mode):
    """The GPU's scale must be one of the oracle's candidates whose error ties the oracle's minimum."""
    s_ref, idx, errs = oracle.grid_scale(W, grid, mode, want_errs=True)
    same = s_gpu == s_ref
    for n in np.nonzero(~same)[0]:
        assert mode == oracle.SCALE_MSE
        amax = np.abs(W[n]).max()
        cands = np.array([np.float32(np.float32(np.float32(100 - i) / np.float32(100) * amax) / grid[3])
                          for i in range(80)])
        hit = np.nonzero(cands == s_gpu[n])[0]
        assert hit.size, "scale is not a candidate of the sweep"
        assert errs[n, hit[0]] <= errs[n].min() * (1 + SUM_RTOL)
    return s_ref, float(same.mean())


@pytest.mark.parametrize("name", ["MNZ_INT", "POT", "SYM", "LLOYD", "NF2", "FAR"])
@pytest.mark.parametrize("N,K", [(37, 4096), (16, 11008), (3, 16384), (5, 20)])
def test_grid_quantize_matches_oracle(name, N, K):
    g = paper_grids()[name]
    W = synth.student_weights(50, N, K) if N % 2 else synth.gaussian_weights(51, N, K)
    W[N // 2] = 0                                                   # an all-zero row keeps scale 1
    for mode in (oracle.SCALE_MSE, oracle.SCALE_ABSMAX):
        s, codes = qift.qift_diag_grid_quantize(dev(W), g, mode)
        s = s.cpu().numpy()
        s_ref, agree = check_scales(W, g, s, mode)
        assert agree > 0.9 and s[N // 2] == 1.0
        if mode == oracle.SCALE_ABSMAX:
            assert np.array_equal(s, s_ref)
        assert np.array_equal(codes.cpu().numpy(), oracle.grid_codes(W, g, s))     # codes at the GPU's own scales
    # given scales, with values planted exactly on the decision boundaries and one ulp above them
    s_ref = oracle.grid_scale(W, g, oracle.SCALE_MSE)[0]
    mids = (g[1:] + g[:-1]) * np.float32(0.5)
    W[0, :3] = mids * s_ref[0]
    W[0, 3:6] = np.nextafter(mids * s_ref[0], np.float32(np.inf))
    s_in = dev(s_ref.copy())
    s_out, codes = qift.qift_diag_grid_quantize(dev(W), g, qift.SCALE_GIVEN, s_n=s_in)
    assert np.array_equal(s_out.cpu().numpy(), s_ref)
    assert np.array_equal(codes.cpu().numpy(), oracle.grid_codes(W, g, s_ref))


def test_grid_quantize_reproduces_the_packer_for_the_no_zero_sets():
    g = paper_grids()
    W = synth.gaussian_weights(52, 48, 4096)
    for key, lv in (("MNZ_INT", qift.MNZ), ("POT", qift.POT)):
        Wd = dev(W)
        packed, s_pack = qift.qift_pack_weights(Wd, lv, qift.SCALE_MSE)
        s, codes = qift.qift_diag_grid_quantize(Wd, g[key], qift.SCALE_GIVEN, s_n=s_pack.clone())
        assert torch.equal(codes, qift.qift_unpack_codes(packed, 48, 4096, lv))


@pytest.mark.parametrize("N,K", [(64, 4096), (7, 11008), (1, 4), (33, 100)])
def test_bucket_stats_match_oracle(N, K):
    g = paper_grids()
    W = synth.gaussian_weights(53, N, K)
    for key in ("MNZ_INT", "SYM", "LLOYD"):
        s = oracle.grid_scale(W, g[key], oracle.SCALE_MSE)[0]
        codes = oracle.grid_codes(W, g[key], s)
        cnt, err = qift.qift_diag_bucket_stats(dev(W), dev(codes), dev(s), g[key])
        cnt_ref, err_ref = oracle.bucket_stats(W, codes, s, g[key])
        assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
        assert np.allclose(err.cpu().numpy(), err_ref, rtol=SUM_RTOL, atol=0)


def test_bucket_stats_sixteen_levels_on_packed_int4():
    N, K = 40, 2048
    W = synth.student_weights(54, N, K)
    Wd = dev(W)
    packed, s = qift.qift_pack_weights(Wd, qift.INT4, qift.SCALE_MSE)
    codes = qift.qift_unpack_codes(packed, N, K, qift.INT4)
    values = [oracle.level_value(oracle.INT4, c) for c in range(16)]
    cnt, err = qift.qift_diag_bucket_stats(Wd, codes, s, values)
    cnt_ref, err_ref = oracle.bucket_stats(W, codes.cpu().numpy(), s.cpu().numpy(), values)
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
    assert np.allclose(err.cpu().numpy(), err_ref, rtol=SUM_RTOL, atol=0)


@pytest.mark.parametrize("n", [1, 2, 31, 1000, 4097, 100_000, 1_300_003])
def test_ratio_scan_matches_oracle(n):
    x = synth.student_t(60, 3, (n,)).astype(np.float32) if n % 2 else synth.normal(61, 3, (n,)).astype(np.float32)
    if n > 40:
        x[5] = 0.0
        x[7] = -x[9]                                                # equal magnitudes
    ratios = [0.005, 0.25, 0.2998, 1 / 3, 0.5, 0.995, 1.0]
    beta, nmse = qift.qift_diag_ratio_scan(dev(x), ratios)
    beta_ref, nmse_ref = oracle.ratio_scan(x, ratios)
    assert np.abs(nmse.cpu().numpy() - nmse_ref).max() <= NMSE_ATOL
    # the minimiser is unique up to ties between splits; where the two sides picked the same split it agrees closely,
    # and in any case the GPU's beta must attain the minimum
    b = beta.cpu().numpy()
    xs = x.astype(np.float64)
    power = (xs ** 2).sum()
    if n <= 100_000:
        for r, bb, e in zip(ratios, b, nmse_ref):
            levels = bb * np.array([-1.0, -r, r, 1.0])
            direct = ((xs[:, None] - levels[None, :]) ** 2).min(1).sum() / power if power > 0 else 0.0
            assert abs(direct - e) <= 10 * NMSE_ATOL
    else:
        assert np.allclose(b, beta_ref, rtol=1e-6)


def test_ratio_scan_full_grid_and_special_inputs():
    x = synth.normal(62, 0, (100_000,)).astype(np.float32)          # the paper's sample count
    grid = np.arange(1, 200) * 0.005
    beta, nmse = qift.qift_diag_ratio_scan(dev(x), grid)
    beta_ref, nmse_ref = oracle.ratio_scan(x, grid)
    assert np.abs(nmse.cpu().numpy() - nmse_ref).max() <= NMSE_ATOL
    assert int(nmse.argmin()) == int(np.argmin(nmse_ref))
    assert np.allclose(beta.cpu().numpy(), beta_ref, rtol=1e-9)
    # all zeros; samples exactly on a grid
    b, e = qift.qift_diag_ratio_scan(dev(np.zeros(100, dtype=np.float32)), [0.3])
    assert float(e[0]) == 0.0 and float(b[0]) == 0.0
    pts = np.float32(0.75) * np.array([-1, -0.3125, 0.3125, 1, 1, -0.3125, 0.3125, 0.3125], dtype=np.float32)
    b, e = qift.qift_diag_ratio_scan(dev(pts), [0.3125])
    assert abs(float(e[0])) <= NMSE_ATOL and abs(float(b[0]) - 0.75) < 1e-7


def test_diag_rejects_bad_arguments():
    W = dev(synth.gaussian_weights(55, 4, 64))
    s = torch.ones(4, device="cuda")
    with pytest.raises(qift.QiftError):
        qift.qift_diag_grid_quantize(W, [1.0, 0.5, 2.0, 3.0], qift.SCALE_MSE)          # not ascending
    with pytest.raises(qift.QiftError):
        qift.qift_diag_grid_quantize(W, [-3.0, -2.0, -1.0, 0.0], qift.SCALE_MSE)        # no positive top level
    codes = torch.zeros((4, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(qift.QiftError):
        qift.qift_diag_bucket_stats(W, codes, s, [0.0, 1.0, 2.0])                       # L must be 4 or 16
    with pytest.raises(qift.QiftError):
        qift.qift_diag_ratio_scan(W.reshape(-1), [0.0])                                 # ratio outside (0, 1]
    with pytest.raises(qift.QiftError):
        qift.qift_diag_ratio_scan(W.reshape(-1), [0.3], workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert qift.qift_diag_ratio_scan_workspace_bytes(0, 1) == 0
    assert qift.qift_diag_ratio_scan_workspace_bytes((1 << 28) + 1, 1) == 0

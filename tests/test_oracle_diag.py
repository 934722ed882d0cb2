"""Pins for the oracle's quantizer diagnostics (CPU only): float four-level grids, the bucket
diagnostic of Sec. 4.5.1 and the ratio scan of Sec. 4.5.2.

Pinned against: the already pinned integer-set quantizer (MNZ and PoT written as float grids give the
same codes, scales and errors), brute-force nearest level, conservation laws of the bucket sums, a
dense brute-force scan over the global scale, the two-level special case r = 1 with its textbook
optimum, samples that lie exactly on a grid, closed forms for a Gaussian source, and the values
the paper prints in Tables 13 and 14.
"""
import numpy as np
import pytest
from scipy import optimize
from scipy.stats import norm

import oracle
import synth
from conftest import read_golden


def paper_grids():
    return {r[0]: np.array([float(v) for v in r[1:]], dtype=np.float32)
            for r in read_golden("level_sets.txt") if r[0] != "RATIO"}


def with_ties(W, grid, s):
    """Plant exact decision-boundary values (midpoints times the scale) into row 0."""
    W = W.copy()
    mids = (grid[1:] + grid[:-1]) * np.float32(0.5)
    W[0, :3] = mids * s[0]
    W[0, 3:6] = np.nextafter(mids * s[0], np.float32(np.inf))
    return W


# ---------------------------------------------------------------------------------- float grids
@pytest.mark.parametrize("name,lv", [("MNZ_INT", oracle.MNZ), ("POT", oracle.POT)])
def test_float_grid_reduces_to_the_integer_sets(name, lv):
    g = paper_grids()[name]
    W = synth.gaussian_weights(11, 9, 768)
    W[4] = 0
    s_i, idx_i, e_i = oracle.weight_scale(W, lv, oracle.SCALE_MSE, want_errs=True)
    s_g, idx_g, e_g = oracle.grid_scale(W, g, oracle.SCALE_MSE, want_errs=True)
    assert np.array_equal(s_i, s_g) and np.array_equal(idx_i, idx_g) and np.array_equal(e_i, e_g)
    s_a, _ = oracle.weight_scale(W, lv, oracle.SCALE_ABSMAX)
    assert np.array_equal(s_a, oracle.grid_scale(W, g, oracle.SCALE_ABSMAX)[0])
    Wt = with_ties(W, g, s_g)
    assert np.array_equal(oracle.grid_codes(Wt, g, s_g), oracle.assign_codes(Wt, lv, s_g))


@pytest.mark.parametrize("name", ["LLOYD", "NF2", "FAR", "SYM"])
def test_float_grid_codes_are_the_nearest_level(name):
    g = paper_grids()[name]
    W = synth.student_weights(12, 6, 640)
    s, idx, errs = oracle.grid_scale(W, g, oracle.SCALE_MSE, want_errs=True)
    codes = oracle.grid_codes(W, g, s)
    t = W / s[:, None]                                                   # fp32 quotient, as defined
    d = np.abs(t.astype(np.float64)[:, :, None] - g.astype(np.float64)[None, None, :])
    brute = d.argmin(2)                                                  # first (lower) level on a tie
    unsure = np.abs(np.sort(d, 2)[:, :, 0] - np.sort(d, 2)[:, :, 1]) < 1e-6
    assert np.array_equal(codes[~unsure], brute[~unsure]) and unsure.mean() < 1e-3
    # the sweep: recompute every candidate's error from the level values alone
    for n in range(W.shape[0]):
        amax = np.abs(W[n]).max()
        for i in (0, 17, 79):
            si = np.float32(np.float32(np.float32(100 - i) / np.float32(100) * amax) / g[3])
            rec = np.float64(si) * g.astype(np.float64)
            e = ((W[n].astype(np.float64)[:, None] - rec[None, :]) ** 2).min(1).sum()
            assert abs(errs[n, i] - e) <= 1e-9 * e
        assert idx[n] == int(np.argmin(errs[n]))
    # exact ties go to the lower level
    Wt = with_ties(W, g, s)
    ct = oracle.grid_codes(Wt, g, s)[0]
    assert list(ct[:3]) == [0, 1, 2] and list(ct[3:6]) == [1, 2, 3]


# ----------------------------------------------------------------------------- bucket diagnostic
def test_bucket_stats_conservation_and_row_errors():
    g = paper_grids()
    W = synth.gaussian_weights(13, 24, 1024)
    for lv, values in ((oracle.MNZ, g["MNZ_INT"]), (oracle.POT, g["POT"]), (oracle.SYM, g["SYM"])):
        s, _ = oracle.weight_scale(W, lv, oracle.SCALE_MSE)
        codes = oracle.assign_codes(W, lv, s)
        cnt, err = oracle.bucket_stats(W, codes, s, values)
        assert cnt.sum() == W.size and np.array_equal(cnt, np.bincount(codes.ravel(), minlength=4))
        rows = sum(oracle.row_sqerr(W[n], lv, float(s[n])) for n in range(W.shape[0]))
        assert abs(err.sum() - rows) <= 1e-12 * rows
    # a planted case with known sums: two rows, every bucket's error written down by hand
    W = np.array([[0.9, -0.1, 0.35, -1.2], [2.0, 2.0, -6.5, 0.0]], dtype=np.float32)
    s = np.array([0.5, 2.0], dtype=np.float32)
    codes = np.array([[3, 1, 2, 0], [2, 2, 0, 1]], dtype=np.uint8)
    values = np.array([-3, -1, 1, 3], dtype=np.float32)
    cnt, err = oracle.bucket_stats(W, codes, s, values)
    w = W.astype(np.float64)
    expect = [(w[0, 3] + 1.5) ** 2 + (w[1, 2] + 6.0) ** 2, (w[0, 1] + 0.5) ** 2 + (w[1, 3] + 2.0) ** 2,
              (w[0, 2] - 0.5) ** 2 + 0.0 + 0.0, (w[0, 0] - 1.5) ** 2]
    assert list(cnt) == [2, 2, 3, 1] and np.allclose(err, expect, rtol=1e-14)


def gaussian_quantizer_stats(levels, s):
    L = np.array(levels, dtype=np.float64) * s
    edges = np.concatenate([[-np.inf], 0.5 * (L[1:] + L[:-1]), [np.inf]])
    a, b = edges[:-1], edges[1:]
    P = norm.cdf(b) - norm.cdf(a)
    with np.errstate(invalid="ignore"):
        pa = np.where(np.isinf(a), 0.0, a * norm.pdf(a))
        pb = np.where(np.isinf(b), 0.0, b * norm.pdf(b))
    m1 = norm.pdf(a) - norm.pdf(b)
    m2 = P + pa - pb
    return P, m2 - 2 * L * m1 + L * L * P


def gaussian_optimum(levels):
    f = lambda s: gaussian_quantizer_stats(levels, s)[1].sum()
    res = optimize.minimize_scalar(f, bounds=(0.05, 3.0), method="bounded", options={"xatol": 1e-10})
    return res.x, res.fun


def test_bucket_stats_reproduce_table13_and_rank_the_float_grids():
    W = synth.normal(77, 0, (192, 4096)).astype(np.float32)
    g = paper_grids()
    paper = {}
    for row in read_golden("table13_buckets.txt"):
        if row[0] != "REL":
            paper.setdefault(row[0], []).append((float(row[2]), float(row[3])))
    total = {}
    for name, key in (("MNZ", "MNZ_INT"), ("POT", "POT"), ("SYM", "SYM"), ("LLOYD", "LLOYD"), ("NF2", "NF2"),
                      ("FAR", "FAR")):
        s, _ = oracle.grid_scale(W, g[key], oracle.SCALE_MSE)
        cnt, err = oracle.bucket_stats(W, oracle.grid_codes(W, g[key], s), s, g[key])
        total[name] = err.sum()
        s_opt, e_opt = gaussian_optimum(g[key])
        P, E = gaussian_quantizer_stats(g[key], s_opt)
        assert np.abs(100.0 * cnt / cnt.sum() - 100 * P).max() < 0.5, name
        assert np.abs(100.0 * err / err.sum() - 100 * E / E.sum()).max() < 0.8, name
        assert abs(err.sum() / W.size - e_opt) < 0.01 * e_opt, name
        if name in paper:
            assert np.abs(100.0 * cnt / cnt.sum() - np.array([p[0] for p in paper[name]])).max() < 0.6
            assert np.abs(100.0 * err / err.sum() - np.array([p[1] for p in paper[name]])).max() < 1.0
    assert total["LLOYD"] < total["MNZ"] < min(total["NF2"], total["POT"])
    assert max(total["NF2"], total["POT"]) < total["SYM"] < total["FAR"]       # no-zero alone is not enough


# ----------------------------------------------------------------------------------- ratio scan
def direct_nmse(x, r, beta):
    """Error of nearest-level quantization onto beta * {-1,-r,r,1}, from the definition."""
    levels = beta * np.array([-1.0, -r, r, 1.0])
    x = x.astype(np.float64)
    return ((x[:, None] - levels[None, :]) ** 2).min(1).sum() / (x ** 2).sum()


@pytest.mark.parametrize("seed,n", [(1, 7), (2, 400), (3, 1500)])
def test_ratio_scan_is_the_minimum_over_the_scale(seed, n):
    x = synth.student_t(seed, 3, (n,)).astype(np.float32)
    ratios = np.array([0.05, 0.25, 1 / 3, 0.5, 0.9])
    beta, nmse = oracle.ratio_scan(x, ratios)
    hi = 2.5 * np.abs(x).max()
    for r, b, e in zip(ratios, beta, nmse):
        assert abs(direct_nmse(x, r, b) - e) <= 1e-12              # the reported scale attains the value
        dense = min(direct_nmse(x, r, bb) for bb in np.linspace(hi / 6000, hi, 6000))
        assert e <= dense + 1e-13 and dense - e < 2e-4             # nothing on a dense grid beats it
        local = [direct_nmse(x, r, b * (1 + d)) for d in (-1e-4, -1e-6, 1e-6, 1e-4)]
        assert min(local) >= e - 1e-13


def test_ratio_scan_special_cases():
    x = synth.normal(5, 0, (5000,)).astype(np.float32)
    a = np.abs(x.astype(np.float64))
    # r = 1 merges inner and outer level: the two-level quantizer {-beta, +beta}, optimum mean|x|
    beta, nmse = oracle.ratio_scan(x, [1.0])
    assert abs(beta[0] - a.mean()) < 1e-12 and abs(nmse[0] - (1 - a.mean() ** 2 / (a ** 2).mean())) < 1e-12
    # samples that sit on a grid are reproduced without error, and the scale is found
    r, b0 = 0.3125, 0.75
    pts = np.float32(b0) * np.array([-1, -r, r, 1, 1, -r, r, r], dtype=np.float32)
    beta, nmse = oracle.ratio_scan(pts, [r])
    assert nmse[0] < 1e-30 and abs(beta[0] - b0) < 1e-12
    # one sample, equal samples, all zeros
    assert oracle.ratio_scan(np.float32([2.5]), [0.3])[1][0] == 0.0
    beta, nmse = oracle.ratio_scan(np.float32([-2.5, 2.5, 2.5]), [0.3])
    assert nmse[0] == 0.0 and beta[0] == 2.5
    assert oracle.ratio_scan(np.zeros(4, dtype=np.float32), [0.3])[1][0] == 0.0
    # the scan does not depend on the order or the signs of the samples
    y = (x * np.where(np.arange(x.size) % 3 == 0, -1, 1).astype(np.float32))[::-1]
    assert np.array_equal(oracle.ratio_scan(x, [0.2, 0.4])[1], oracle.ratio_scan(y, [0.2, 0.4])[1])
    # scale covariance: x -> c x leaves NMSE alone and multiplies beta by c (c a power of two: exact)
    b1, n1 = oracle.ratio_scan(x, [0.3])
    b2, n2 = oracle.ratio_scan(x * np.float32(4), [0.3])
    assert abs(n1[0] - n2[0]) < 1e-14 and abs(b2[0] - 4 * b1[0]) < 1e-12


def test_ratio_scan_reproduces_table14():
    paper = {r[0]: (float(r[1]), float(r[2])) for r in read_golden("table14_ratio_nmse.txt")}
    x = synth.normal(78, 0, (1 << 20,)).astype(np.float32)
    names = ["LLOYD", "MNZ", "NF2", "POT", "FAR"]
    ratios = [0.4528 / 1.5104, 1 / 3, 0.2525685, 0.25, 0.5]
    beta, nmse = oracle.ratio_scan(x, ratios)
    for name, r, b, e in zip(names, ratios, beta, nmse):
        s_opt, closed = gaussian_optimum(np.array([-1, -r, r, 1.0]))
        assert abs(e - closed) < 0.004 * closed                    # sampling noise of 1M samples
        assert abs(b - s_opt) < 0.01 * s_opt
        assert abs(e - paper[name][1]) < 0.01 * paper[name][1]     # real weights are near-Gaussian
        assert abs(r - paper[name][0]) < 6e-5
    assert list(np.argsort(nmse)) == [0, 1, 2, 3, 4]               # the table's ordering
    # the 0.005 grid: the best ratio is 0.30 and it is NMSE-equivalent to Lloyd-Max
    grid = np.arange(1, 200) * 0.005
    _, scan = oracle.ratio_scan(x, grid)
    best = int(np.argmin(scan))
    assert abs(grid[best] - paper["SCAN_BEST"][0]) <= 0.005 + 1e-12
    assert abs(scan[best] - nmse[0]) < 2e-6
    assert abs(scan[best] - paper["SCAN_BEST"][1]) < 0.01 * paper["SCAN_BEST"][1]

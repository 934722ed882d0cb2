"""Pins for the KV4 part of the oracle (Sec. 4.1: asymmetric 4-bit keys and values, clipping ratio 0.95).

None of these re-types the oracle's formula: they are brute force over the 16 levels, closed-form special
cases, invariants of softmax attention, and a library routine (scipy's softmax) on the dequantized cache."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle
import synth


def rows(seed, n, D, shift=0.0, scale=1.0):
    return (synth.normal(seed, 7, (n, D)) * scale + shift).astype(np.float32)


def dequant(codes, s, z):
    return s[..., None].astype(np.float64) * (codes.astype(np.float64) - z[..., None].astype(np.float64))


def test_codes_are_the_nearest_of_the_sixteen_levels():
    # brute force: inside the clipped range the chosen code is the level closest to x (fp64, away from ties)
    X = rows(11, 64, 128, shift=0.3)
    codes, s, z = oracle.kv4_quantize(X, 0, 0.95)
    levels = s[:, None, None].astype(np.float64) * (np.arange(16)[None, None, :] - z[:, None, None].astype(np.float64))
    dist = np.abs(X[:, :, None].astype(np.float64) - levels)
    best = dist.argmin(axis=2)
    srt = np.sort(dist, axis=2)
    clear = (srt[:, :, 1] - srt[:, :, 0]) > 1e-6 * s[:, None]
    assert clear.mean() > 0.99
    assert np.array_equal(codes[clear], best[clear].astype(np.uint8))
    assert codes.min() == 0 and codes.max() == 15 and set(np.unique(z)) <= set(range(16))


def test_zero_is_a_level_and_error_is_half_a_step_inside_the_range():
    X = rows(12, 32, 128, shift=-0.2, scale=2.0)
    X[:, 5] = 0.0
    codes, s, z = oracle.kv4_quantize(X, 0, 0.95)
    xh = dequant(codes, s, z)
    assert np.all(xh[:, 5] == 0.0) and np.all(codes[:, 5] == z)                 # x = 0 -> code z -> exactly 0
    lo = s * (0 - z)
    hi = s * (15 - z)
    inside = (X >= lo[:, None]) & (X <= hi[:, None])
    assert np.all(np.abs(xh - X)[inside] <= 0.5 * s[:, None].repeat(128, 1)[inside] * (1 + 1e-5))
    assert np.all(codes[X > hi[:, None]] == 15) and np.all(codes[X < lo[:, None]] == 0)   # clipped tails saturate


def test_range_follows_the_clipping_ratio():
    X = rows(13, 16, 128)
    for clip in (1.0, 0.95, 0.5):
        codes, s, z = oracle.kv4_quantize(X, 0, clip)
        want = (clip * (X.max(1).astype(np.float64) - X.min(1).astype(np.float64))) / 15.0
        assert np.allclose(s, want, rtol=1e-6)
    codes, s, z = oracle.kv4_quantize(X, 0, 1.0)                                 # nothing clipped: extremes hit the end codes
    assert np.all(codes[np.arange(16), X.argmax(1)] == 15) and np.all(codes[np.arange(16), X.argmin(1)] == 0)


def test_one_sided_and_constant_rows():
    pos = np.abs(rows(14, 4, 64)) + 0.1
    codes, s, z = oracle.kv4_quantize(pos, 0, 0.95)
    assert np.all(z == 0) and np.allclose(s, 0.95 * pos.max(1) / 15.0, rtol=1e-6)  # range starts at zero
    codes, s, z = oracle.kv4_quantize(-pos, 0, 0.95)
    assert np.all(z == 15)
    codes, s, z = oracle.kv4_quantize(np.zeros((3, 64), np.float32), 0, 0.95)
    assert np.all(s == 1.0) and np.all(z == 0) and np.all(codes == 0)


def test_rotation_is_orthonormal_and_spreads_an_outlier():
    X = rows(15, 8, 128)
    X[:, 7] += 40.0                                                              # one outlier channel
    c0, s0, z0 = oracle.kv4_quantize(X, 0, 1.0)
    c1, s1, z1 = oracle.kv4_quantize(X, 128, 1.0)
    # rotated rows have the same norm: compare the dequantized norms with the input's, and the step is much finer
    n_in = np.linalg.norm(X.astype(np.float64), axis=1)
    n_rot = np.linalg.norm(dequant(c1, s1, z1), axis=1)
    assert np.allclose(n_rot, n_in, rtol=2e-2)
    assert np.all(s1 < 0.5 * s0)
    # dequantized rotated row, rotated back with the closed-form matrix, is closer to x than the unrotated code
    H = np.array([[(-1) ** bin(i & j).count("1") for j in range(128)] for i in range(128)], dtype=np.float64) / np.sqrt(128)
    back = dequant(c1, s1, z1) @ H
    assert np.linalg.norm(back - X) < 0.5 * np.linalg.norm(dequant(c0, s0, z0) - X)


def test_pack_roundtrip_and_nibble_order():
    codes = (np.arange(2 * 3 * 64) % 16).astype(np.uint8).reshape(2, 3, 64)
    packed = oracle.kv4_pack(codes)
    assert packed.shape == (2, 3, 32) and packed.dtype == np.uint8
    assert np.array_equal(oracle.kv4_unpack(packed), codes)
    assert packed[0, 0, 0] == (codes[0, 0, 0] | (codes[0, 0, 1] << 4))           # even dimension in the low nibble


def test_token_pair_packing_of_values():
    codes = ((np.arange(2 * 6 * 64).reshape(2, 6, 64) * 7) % 16).astype(np.uint8)
    packed = oracle.kv4_pack_token_pairs(codes)
    assert packed.shape == (2, 3, 64)
    assert np.array_equal(packed & 15, codes[:, 0::2]) and np.array_equal(packed >> 4, codes[:, 1::2])


def make_cache(seed, Hkv, T, D):
    K = rows(seed, Hkv * T, D, shift=0.1)
    V = rows(seed + 1, Hkv * T, D, shift=-0.1)
    kc, ks, kz = oracle.kv4_quantize(K, 0, 0.95)
    vc, vs, vz = oracle.kv4_quantize(V, 0, 0.95)
    sh = (Hkv, T)
    return kc.reshape(Hkv, T, D), ks.reshape(sh), kz.reshape(sh), vc.reshape(Hkv, T, D), vs.reshape(sh), vz.reshape(sh)


def test_attention_against_scipy_softmax_on_the_dequantized_cache():
    Hq, Hkv, T, D = 8, 2, 37, 64
    kc, ks, kz, vc, vs, vz = make_cache(20, Hkv, T, D)
    q = rows(22, Hq, D)
    out = oracle.kv4_attention(q, kc, ks, kz, vc, vs, vz)
    Kh, Vh = dequant(kc, ks, kz), dequant(vc, vs, vz)
    for h in range(Hq):
        kv = h // (Hq // Hkv)                                                    # grouped queries share a KV head
        p = softmax(Kh[kv] @ q[h].astype(np.float64) / np.sqrt(D))
        assert np.allclose(out[h], p @ Vh[kv], rtol=1e-12, atol=1e-14)


def test_attention_special_cases():
    Hq, Hkv, T, D = 4, 4, 9, 64
    kc, ks, kz, vc, vs, vz = make_cache(30, Hkv, T, D)
    Vh = dequant(vc, vs, vz)
    q = rows(32, Hq, D)
    # one cached token: the output is that token's value
    out1 = oracle.kv4_attention(q, kc[:, :1], ks[:, :1], kz[:, :1], vc[:, :1], vs[:, :1], vz[:, :1])
    assert np.allclose(out1, Vh[:, 0], rtol=1e-13)
    # zero query: uniform weights, the mean of the values
    out0 = oracle.kv4_attention(np.zeros_like(q), kc, ks, kz, vc, vs, vz)
    assert np.allclose(out0, Vh.mean(axis=1), rtol=1e-12)
    # identical keys: uniform again, whatever the query
    kc2 = np.repeat(kc[:, :1], T, axis=1)
    outu = oracle.kv4_attention(q, kc2, np.repeat(ks[:, :1], T, 1), np.repeat(kz[:, :1], T, 1), vc, vs, vz)
    assert np.allclose(outu, Vh.mean(axis=1), rtol=1e-12)
    # order of the cached tokens does not matter
    perm = np.random.default_rng(0).permutation(T)
    outp = oracle.kv4_attention(q, kc[:, perm], ks[:, perm], kz[:, perm], vc[:, perm], vs[:, perm], vz[:, perm])
    assert np.allclose(outp, oracle.kv4_attention(q, kc, ks, kz, vc, vs, vz), rtol=1e-12)
    # the output is a convex combination of the values
    out = oracle.kv4_attention(q, kc, ks, kz, vc, vs, vz)
    assert np.all(out <= Vh.max(axis=1) + 1e-12) and np.all(out >= Vh.min(axis=1) - 1e-12)
    # a query that matches one key overwhelmingly returns that token's value
    big = (dequant(kc, ks, kz)[:, 3] * 50.0).astype(np.float32)
    outb = oracle.kv4_attention(big, kc, ks, kz, vc, vs, vz)
    assert np.allclose(outb, Vh[:, 3], atol=1e-6)

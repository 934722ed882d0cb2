"""KV4 cache path on the GPU against the oracle: the quantizer bit-exactly (codes, scales, zero-points), the decode
attention within the fp32 tolerance derived below."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift

pytestmark = pytest.mark.gpu
D = 128
# Tolerance of the attention output: the kernel works in fp32 (128-term dot products, expf, running sums over T
# tokens), the oracle in fp64.  A score carries an absolute error of a few 1e-6 * |score| (|score| <= ~30 here), which
# exp turns into the same RELATIVE error of each weight; the normalised output, a convex combination of values, is then
# off by a few 1e-5 of the largest |value|.  Bound used: 2e-4 * max|V|.
ATOL_FRAC = 2e-4


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def vectors(seed, T, H, shift, outlier=None):
    x = (synth.normal(seed, 3, (T, H, D)) + shift).astype(np.float32)
    if outlier is not None:
        x[:, :, outlier] *= 12.0
    return x


@pytest.mark.parametrize("had_block", [0, 128, 16])
@pytest.mark.parametrize("bf16", [False, True])
def test_kv4_quantize_keys_matches_oracle(had_block, bf16):
    T, H = 37, 5
    x = vectors(40, T, H, 0.2, outlier=9)
    xd = dev(x)
    if bf16:
        xd = xd.to(torch.bfloat16)
        x = oracle.bf16_to_f32(xd.view(torch.int16).cpu().numpy().view(np.uint16)).reshape(T, H, D)
    cache = qift.Kv4Cache(H, 64)
    qift.qift_kv4_quantize(xd, cache, t0=3, had_block=had_block, clip_ratio=0.95)
    codes, s, z = oracle.kv4_quantize(x.reshape(T * H, D), had_block, 0.95)
    packed = oracle.kv4_pack(codes).reshape(T, H, D // 2).transpose(1, 0, 2)      # head-major like the cache
    assert np.array_equal(cache.codes.cpu().numpy()[:, 3:3 + T], packed)
    assert np.array_equal(cache.scale.cpu().numpy()[:, 3:3 + T], s.reshape(T, H).T)
    assert np.array_equal(cache.zero.cpu().numpy()[:, 3:3 + T], z.reshape(T, H).T)
    assert not cache.codes.cpu().numpy()[:, :3].any() and not cache.codes.cpu().numpy()[:, 3 + T:].any()
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK


@pytest.mark.parametrize("t0,T", [(0, 36), (3, 37), (4, 1), (5, 1), (7, 2)])
def test_kv4_quantize_values_token_pairs(t0, T):
    # the value cache holds two consecutive tokens per byte: appends of any parity must keep the partner nibble
    H, T_cap = 3, 64
    cache = qift.Kv4Cache(H, T_cap, qift.KV_VALUES)
    ref_codes = np.zeros((H, T_cap, D), np.uint8)
    ref_s = np.zeros((H, T_cap), np.float32)
    ref_z = np.zeros((H, T_cap), np.float32)
    pos = 0
    for step, (a, n) in enumerate([(0, t0), (t0, T)]):                            # fill [0, t0) first, then append T tokens
        if n == 0:
            continue
        x = vectors(41 + step, n, H, -0.3)
        qift.qift_kv4_quantize(dev(x), cache, t0=a, had_block=0, clip_ratio=0.95)
        codes, s, z = oracle.kv4_quantize(x.reshape(n * H, D), 0, 0.95)
        ref_codes[:, a:a + n] = codes.reshape(n, H, D).transpose(1, 0, 2)
        ref_s[:, a:a + n] = s.reshape(n, H).T
        ref_z[:, a:a + n] = z.reshape(n, H).T
    assert np.array_equal(cache.codes.cpu().numpy(), oracle.kv4_pack_token_pairs(ref_codes))
    assert np.array_equal(cache.scale.cpu().numpy(), ref_s) and np.array_equal(cache.zero.cpu().numpy(), ref_z)


def test_kv4_quantize_degenerate_rows():
    x = np.zeros((4, 2, D), np.float32)
    x[1] = 3.0                      # constant positive: range [0, 3]
    x[2] = -2.0                     # constant negative
    x[3, :, 0] = 1e-30              # tiny range
    cache = qift.Kv4Cache(2, 4)
    qift.qift_kv4_quantize(dev(x), cache)
    codes, s, z = oracle.kv4_quantize(x.reshape(8, D), 0, 0.95)
    assert np.array_equal(cache.codes.cpu().numpy(), oracle.kv4_pack(codes).reshape(4, 2, D // 2).transpose(1, 0, 2))
    assert np.array_equal(cache.scale.cpu().numpy(), s.reshape(4, 2).T)
    assert np.array_equal(cache.zero.cpu().numpy(), z.reshape(4, 2).T)


def build_cache(seed, T, Hkv, T_cap):
    k = vectors(seed, T, Hkv, 0.1, outlier=5)
    v = vectors(seed + 1, T, Hkv, -0.1)
    T_cap += T_cap & 1
    K, V = qift.Kv4Cache(Hkv, T_cap), qift.Kv4Cache(Hkv, T_cap, qift.KV_VALUES)
    qift.qift_kv4_quantize(dev(k), K, had_block=128)
    qift.qift_kv4_quantize(dev(v), V, had_block=0)
    kc = oracle.kv4_unpack(K.codes.cpu().numpy()[:, :T])
    vb = V.codes.cpu().numpy()                                                    # [Hkv, T_cap/2, D]: tokens 2i | 2i+1 << 4
    vc = np.stack([vb & 15, vb >> 4], axis=2).reshape(Hkv, T_cap, D)[:, :T]
    return K, V, (kc, K.scale.cpu().numpy()[:, :T], K.zero.cpu().numpy()[:, :T],
                  vc, V.scale.cpu().numpy()[:, :T], V.zero.cpu().numpy()[:, :T])


@pytest.mark.parametrize("T,Hq,Hkv", [(1, 4, 4), (5, 8, 2), (16, 6, 2), (130, 8, 8), (1000, 32, 8), (4133, 32, 8),
                                      (3000, 16, 2), (999, 14, 2), (20000, 8, 8)])
def test_kv4_attention_matches_oracle(T, Hq, Hkv):
    K, V, ref_args = build_cache(50 + T, T, Hkv, T + 11)
    q = (synth.normal(60, 4, (Hq, D)) * 1.5).astype(np.float32)
    out = qift.qift_kv4_attention_decode(dev(q), K, V, T).cpu().numpy()
    ref = oracle.kv4_attention(q, *ref_args)
    vmax = np.abs(ref_args[4][..., None] * (ref_args[3].astype(np.float64) - ref_args[5][..., None])).max()
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() <= ATOL_FRAC * vmax
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK


def test_kv4_attention_ignores_unwritten_slots():
    """Slots T .. T_cap-1 have not been written yet; whatever they hold (NaN scales included) must not reach the output."""
    T, Hq, Hkv = 1000, 8, 2
    K, V, ref_args = build_cache(80, T, Hkv, T + 40)
    q = (synth.normal(81, 4, (Hq, D)) * 1.5).astype(np.float32)
    ref = oracle.kv4_attention(q, *ref_args)
    for c in (K, V):
        c.scale[:, T:] = float("nan")
        c.zero[:, T:] = float("inf")
    K.codes[:, T:] = 0xFF
    V.codes[:, (T + 1) // 2:] = 0xFF
    out = qift.qift_kv4_attention_decode(dev(q), K, V, T).cpu().numpy()
    vmax = np.abs(ref_args[4][..., None] * (ref_args[3].astype(np.float64) - ref_args[5][..., None])).max()
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() <= ATOL_FRAC * vmax


def test_kv4_attention_peaked_and_uniform_scores():
    T, Hq, Hkv = 700, 4, 4
    K, V, ref_args = build_cache(70, T, Hkv, T)
    kc, ks, kz = ref_args[:3]
    khat = ks[..., None] * (kc.astype(np.float64) - kz[..., None])
    peaked = (khat[:, 123] * 6.0).astype(np.float32)          # scores dominated by one token (large exponents)
    for q in (peaked, np.zeros((Hq, D), np.float32)):
        out = qift.qift_kv4_attention_decode(dev(q), K, V, T).cpu().numpy()
        ref = oracle.kv4_attention(q, *ref_args)
        vmax = np.abs(ref_args[4][..., None] * (ref_args[3].astype(np.float64) - ref_args[5][..., None])).max()
        assert np.abs(out - ref).max() <= ATOL_FRAC * vmax


def test_kv4_rejects_bad_arguments():
    L = qift.lib()
    with pytest.raises(AssertionError):
        qift.Kv4Cache(2, 15)                                                      # odd capacity
    K = qift.Kv4Cache(2, 16)
    x = torch.zeros((4, 2, 64), device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_kv4_quantize(x, K)                                              # D != 128
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    x = torch.zeros((17, 2, D), device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_kv4_quantize(x, K)                                              # more tokens than slots
    assert e.value.status == qift.ERR_INVALID_ARG
    q = torch.zeros((18, D), device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_kv4_attention_decode(q, K, K, 4)                                # 9 query heads per KV head
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    q = torch.zeros((4, D), device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_kv4_attention_decode(q, K, K, 4, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == qift.ERR_WORKSPACE
    assert L.qift_kv4_attention_workspace_bytes(0, 4, 2) == 0

"""Pins for the oracle's Hadamard rotation and activation quantizer (CPU only).

Each check compares the oracle with something that is not the oracle: the closed form
H[i][j] = (-1)^popcount(i & j), exact integer identities, a brute-force nearest-integer search,
or values fixed by the paper (clip ratio 0.9, INT4 range of Eq. 1).
"""
import numpy as np
import pytest

import oracle
import synth


def dense_hadamard(B):
    i = np.arange(B)
    pc = np.zeros((B, B), dtype=np.int64)
    a = i[:, None] & i[None, :]
    while a.any():
        pc += a & 1
        a >>= 1
    return 1 - 2 * (pc & 1)


@pytest.mark.parametrize("B", [2, 4, 8, 64, 256, 1024, 4096])
def test_butterfly_is_sylvester_matrix(B):
    # the oracle's transform of the unit vectors IS the matrix: compare entry by entry, in integers
    if B <= 1024:
        H = oracle.wht_blocks(np.eye(B, dtype=np.float32), B)
        Hd = dense_hadamard(B)
        assert np.array_equal(H.astype(np.int64), Hd)
        assert np.array_equal(Hd, Hd.T)                                   # symmetric
        assert np.array_equal(Hd @ Hd.T, B * np.eye(B, dtype=np.int64))   # H H^T = B I
    else:
        rows = [0, 1, 2, 3, 1023, 2048, 4095, 2730]
        e = np.zeros((len(rows), B), dtype=np.float32)
        e[np.arange(len(rows)), rows] = 1
        H = oracle.wht_blocks(e, B).astype(np.int64)
        Hd = dense_hadamard(B)[rows]
        assert np.array_equal(H, Hd)
        assert np.array_equal(H @ H.T, B * np.eye(len(rows), dtype=np.int64))


@pytest.mark.parametrize("B,K", [(256, 256), (256, 11008), (2048, 14336), (4096, 4096)])
def test_butterfly_matches_dense_matvec(B, K):
    x = synth.normal(11, 0, (3, K)).astype(np.float32)
    u = oracle.wht_blocks(x, B).astype(np.float64)
    Hd = dense_hadamard(B).astype(np.float64)
    ref = (x.astype(np.float64).reshape(3, K // B, B) @ Hd).reshape(3, K)
    bound = B * 2.0 ** -23 * np.abs(x).max() * 4
    assert np.abs(u - ref).max() <= bound
    # Parseval and involution
    assert np.allclose((u ** 2).sum(1), B * (x.astype(np.float64) ** 2).sum(1), rtol=1e-5)
    uu = oracle.wht_blocks(u.astype(np.float32), B)
    assert np.allclose(uu, B * x, rtol=0, atol=B * np.abs(x).max() * 1e-5)


def test_special_vectors():
    B = 512
    e0 = np.zeros((1, B), dtype=np.float32)
    e0[0, 0] = 1
    assert np.array_equal(oracle.wht_blocks(e0, B), np.ones((1, B), dtype=np.float32))
    ones = np.ones((1, B), dtype=np.float32)
    out = oracle.wht_blocks(ones, B)
    assert out[0, 0] == B and not out[0, 1:].any()
    # blocks are independent: transforming K = 2B equals transforming each half
    x = synth.normal(5, 0, (1, 2 * B)).astype(np.float32)
    whole = oracle.wht_blocks(x, B)
    halves = np.concatenate([oracle.wht_blocks(x[:, :B], B), oracle.wht_blocks(x[:, B:], B)], 1)
    assert np.array_equal(whole, halves)
    # a sign error in the butterfly (a-b vs b-a) would break this one: H e1 = (+,-,+,-,...)
    e1 = np.zeros((1, 8), dtype=np.float32)
    e1[0, 1] = 1
    assert np.array_equal(oracle.wht_blocks(e1, 8)[0], np.array([1, -1] * 4, dtype=np.float32))


def test_rotation_preserves_the_product():
    # (W Q)(Q x) = W x: the rotation is orthogonal, so the layer output is unchanged
    N, K, B = 16, 1024, 256
    W = synth.student_weights(3, N, K)
    x = synth.normal(4, 0, (1, K)).astype(np.float32)
    Wr = oracle.rotate_weights(W, B).astype(np.float64)
    xr = oracle.rotate_weights(x, B).astype(np.float64)
    ref = W.astype(np.float64) @ x.astype(np.float64).T
    got = Wr @ xr.T
    assert np.abs(got - ref).max() <= 1e-5 * np.abs(ref).max() + 1e-6
    # and Q is orthonormal: rows keep their norm
    assert np.allclose((Wr ** 2).sum(1), (W.astype(np.float64) ** 2).sum(1), rtol=1e-5)


def test_outlier_diffusion():
    B = 256
    spike = np.zeros((1, B), dtype=np.float32)
    spike[0, 37] = 20.0
    r = oracle.rotate_weights(spike, B)
    assert np.allclose(np.abs(r), 20.0 / 16.0)
    # config-1 style row: 4 outlier channels x20 -> the rotated maximum is far below the raw one
    x, ch = synth.activations(7, 1, B, 4)
    xr = oracle.rotate_weights(x, B)
    assert len(ch) == 4
    assert np.abs(xr).max() < 0.5 * np.abs(x).max()


def test_student_t_weights_become_gaussian_like():
    # heavy-tailed stand-in: excess kurtosis ~6 before, ~6/K after rotation (cf. Table 3)
    N, K = 64, 4096
    W = synth.student_weights(9, N, K)
    Wr = oracle.rotate_weights(W, K)

    def kurt(a):
        z = (a - a.mean(1, keepdims=True)) / a.std(1, keepdims=True)
        return np.abs((z ** 4).mean(1) - 3).mean()

    assert kurt(W.astype(np.float64)) > 1.0
    assert kurt(Wr.astype(np.float64)) < 0.2


@pytest.mark.parametrize("B", [0, 256])
@pytest.mark.parametrize("clip", [0.9, 1.0])
def test_act_quant_is_eq1_with_b4(B, clip):
    M, K = 5, 512
    x, _ = synth.activations(21, M, K, 5)
    q, s_a = oracle.quantize_act(x, B, clip)
    u = oracle.wht_blocks(x, B).astype(np.float64) if B else x.astype(np.float64)
    amax = np.abs(u).max(1)
    norm = np.sqrt(B) if B else 1.0
    # scale: clip*amax maps to +7; the 1/sqrt(B) of the orthonormal rotation sits in s_a
    s_u = s_a.astype(np.float64) * norm
    assert np.allclose(s_u, clip * amax / 7.0, rtol=3e-7)
    # brute force: q is the integer of [-8, 7] nearest to u / s_u
    t = u / s_u[:, None]
    cand = np.arange(-8, 8)[None, None, :]
    dist = np.abs(t[:, :, None] - cand)
    best = dist.min(2)
    chosen = np.abs(t - q)
    near_tie = np.abs(np.abs(t - np.floor(t)) - 0.5) < 1e-5
    assert np.all((chosen <= best + 1e-6) | near_tie)
    assert q.min() >= -8 and q.max() <= 7
    # unclipped entries reconstruct to within half a step
    inside = np.abs(t) <= 7
    assert np.all(np.abs(u - q * s_u[:, None])[inside] <= 0.5 * s_u.max() * (1 + 1e-6))
    # the arg-max element lands on +7 (or -8 for a negative one when clip < 1: 7/0.9 = 7.78 -> -8)
    for m in range(M):
        k = np.abs(u[m]).argmax()
        if clip == 1.0:
            assert abs(q[m, k]) == 7
        else:
            assert q[m, k] == (7 if u[m, k] > 0 else -8)


def test_act_quant_ties_and_zero_row():
    # s_u = 0.9*7/7... build a row whose scale is exactly 1: amax*clip/7 = 1 with clip = 1, amax = 7
    x = np.array([[7.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 6.5]], dtype=np.float32)
    q, s = oracle.quantize_act(x, 0, 1.0)
    assert s[0] == 1.0
    assert q[0].tolist() == [7, 0, 2, 2, 0, -2, -2, 6]      # round half to even
    z = np.zeros((2, 16), dtype=np.float32)
    q, s = oracle.quantize_act(z, 16, 0.9)
    assert not q.any() and np.all(s == np.float32(1.0) * np.float32(0.25))
    # -8 is reachable, +8 is not
    x = np.array([[-10.0, 10.0, 0, 0]], dtype=np.float32)
    q, s = oracle.quantize_act(x, 0, 0.9)
    assert q[0].tolist() == [-8, 7, 0, 0]


def test_bf16_roundtrip_helpers():
    import torch
    x = synth.normal(2, 0, (4096,)).astype(np.float32) * 3
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]   # exact ties at the bf16 boundary
    got = oracle.f32_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, ref)
    # integer definition of round-to-nearest-even
    u = x.view(np.uint32).astype(np.uint64)
    man = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    assert np.array_equal(got, man)
    back = oracle.bf16_to_f32(got)
    assert np.array_equal(back.view(np.uint32), got.astype(np.uint32) << 16)


# ------------------------------------------------------------------------------- full-dimension rotation, K = 28 * 2^p
def sylvester(P):
    return np.array([[(-1) ** bin(i & j).count("1") for j in range(P)] for i in range(P)], dtype=np.int64)


def test_hadamard28_is_a_symmetric_hadamard_matrix():
    H = oracle.hadamard28().astype(np.int64)
    assert set(np.unique(H)) == {-1, 1}
    assert np.array_equal(H @ H.T, 28 * np.eye(28, dtype=np.int64))     # closed form of a Hadamard matrix
    assert np.array_equal(H, H.T)                                        # Paley II with q = 1 mod 4 is symmetric
    # the conference core: first row / column of the top-left block C + I are all ones
    assert np.all(H[0, :14] == 1) and np.all(H[:14, 0] == 1)


@pytest.mark.parametrize("P", [1, 4, 16])
def test_kron28_rotation_against_the_dense_kronecker_product(P):
    K = 28 * P
    H = np.kron(oracle.hadamard28().astype(np.int64), sylvester(P))      # block index outer, position inner
    assert np.array_equal(H @ H.T, K * np.eye(K, dtype=np.int64))
    x = synth.normal(77, 1, (3, K)).astype(np.float32)
    got = oracle.rotate_weights(x, K).astype(np.float64) * np.sqrt(K)    # undo the orthonormal factor
    want = x.astype(np.float64) @ H.T
    assert np.allclose(got, want, rtol=0, atol=K * 2.0 ** -22 * np.abs(x).max())
    # orthonormal and symmetric: applying it twice gives the input back
    back = oracle.rotate_weights(oracle.rotate_weights(x, K), K)
    assert np.allclose(back, x, atol=1e-5)


def test_kron28_quantizer_uses_the_full_dimension_scale():
    K = 28 * 16
    x = synth.normal(78, 1, (2, K)).astype(np.float32)
    x[:, 5] += 50.0                                                      # one outlier channel: spread over all K
    q, s = oracle.quantize_act(x, K, 0.9)
    qb, sb = oracle.quantize_act(x, 16, 0.9)                             # block-diagonal alternative
    assert q.min() >= -8 and q.max() <= 7
    u = oracle.rotate_weights(x, K).astype(np.float64)                   # orthonormal rotation of the row
    assert np.allclose(s.astype(np.float64) * 7 / 0.9, np.abs(u).max(axis=1), rtol=1e-5)
    assert np.all(s < 0.5 * sb)                                          # the outlier is diffused much further

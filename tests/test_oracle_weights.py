"""Pins for the oracle's weight quantizer, packer, integer product and epilogue (CPU only).

Pinned against: the level sets and ratios the paper prints (text fixtures under golden/), the
identities of Sec. 3.3 (half-scale form, z = 1.5 form), Eq. 1, brute-force nearest level and
brute-force enumeration of the product, and closed forms for a Gaussian source (the paper's own
source model) that reproduce Tables 13 and 14.
"""
import itertools

import numpy as np
import pytest
from scipy import optimize
from scipy.stats import norm

import oracle
import synth
from conftest import read_golden

LV = {"MNZ": oracle.MNZ, "POT": oracle.POT, "SYM": oracle.SYM}


def paper_levels():
    out = {}
    for row in read_golden("level_sets.txt"):
        if row[0] != "RATIO":
            out[row[0]] = [float(v) for v in row[1:]]
    return out


# ----------------------------------------------------------------------------- level sets (P5, P6)
def test_level_tables_match_the_paper():
    g = paper_levels()
    assert oracle.level_table(oracle.SYM) == g["SYM"]
    assert oracle.level_table(oracle.POT) == g["POT"]
    assert oracle.level_table(oracle.MNZ) == g["MNZ_INT"]
    # half-scale identity: {-1.5,-.5,.5,1.5} s == {-3,-1,1,3} (s/2), exactly in fp32
    for s in np.float32([0.013, 1.0, 7.25e-4]):
        full = np.float32(g["MNZ"]) * s
        half = np.float32(oracle.level_table(oracle.MNZ)) * (np.float32(0.5) * s)
        assert np.array_equal(full, half)
    # zero-point form: s (q - 1.5), q = 0..3, doubled, is the stored integer level of code q
    assert [int(2 * (q - 1.5)) for q in range(4)] == oracle.level_table(oracle.MNZ)
    # mirror sets: L[c] = -L[3-c]; the standard set is not a mirror set and contains zero
    for lv in (oracle.MNZ, oracle.POT):
        t = oracle.level_table(lv)
        assert all(t[c] == -t[3 - c] for c in range(4)) and 0 not in t
    t = oracle.level_table(oracle.SYM)
    assert 0 in t and any(t[c] != -t[3 - c] for c in range(4))
    # INT4 is Eq. 1's range -8..7 in two's complement
    assert sorted(oracle.level_table(oracle.INT4)) == list(range(-8, 8))
    assert all(((v + 16) & 15) == c for c, v in enumerate(oracle.level_table(oracle.INT4)))
    # INT3 (the W3A4 configuration of Sec. 4.4) is Eq. 1's range for b = 3, -2^(b-1) .. 2^(b-1) - 1, in two's complement
    assert sorted(oracle.level_table(oracle.INT3)) == list(range(-(2 ** 2), 2 ** 2))
    assert all(((v + 8) & 7) == c for c, v in enumerate(oracle.level_table(oracle.INT3)))
    # plane form used by the storage: level = (code & 3) - 4 (code >> 2)
    assert all(oracle.level_value(oracle.INT3, c) == (c & 3) - 4 * (c >> 2) for c in range(8))


def test_inner_outer_ratio_is_scale_invariant():
    ratios = {r[1]: float(r[2]) for r in read_golden("level_sets.txt") if r[0] == "RATIO"}
    for name, lv, mult in (("MNZ", oracle.MNZ, 3), ("POT", oracle.POT, 4)):
        t = oracle.level_table(lv)
        assert mult * t[2] == t[3] and mult * t[1] == t[0]          # in integers
        for s in (1e-3, 0.37, 12.5):
            assert abs((t[2] * s) / (t[3] * s) - 1.0 / mult) < 1e-15
        assert abs(1.0 / mult - ratios[name]) < 5e-5


def test_affine_bit_plane_identity():
    # every set is affine in the two code bits: level = a*b1 + b*b0 + c
    for lv, (a, b, c) in ((oracle.MNZ, (4, 2, -3)), (oracle.POT, (5, 3, -4)), (oracle.SYM, (2, 1, -2))):
        for code in range(4):
            assert oracle.level_value(lv, code) == a * (code >> 1) + b * (code & 1) + c


# ----------------------------------------------------------------------------- nearest level (P7)
@pytest.mark.parametrize("name", ["MNZ", "POT", "SYM", "INT4", "INT3"])
def test_nearest_level_brute_force(name):
    lv = getattr(oracle, name)
    table = np.array(oracle.level_table(lv), dtype=np.float64)
    s = np.float32(0.0173)
    top = table.max()
    t = np.concatenate([np.linspace(-1.5 * top - 2, 1.5 * top + 2, 20001), synth.normal(1, 0, (20000,)) * 2])
    w = (t * s).astype(np.float32)[None, :]
    codes = oracle.assign_codes(w, lv, np.array([s]))[0]
    tt = w[0].astype(np.float64) / np.float64(s)
    dist = np.abs(tt[:, None] - table[None, :])
    best = dist.min(1)
    chosen = dist[np.arange(len(tt)), codes]
    second = np.sort(dist, 1)[:, 1]
    clear = (second - best) > 1e-4           # away from decision thresholds
    assert np.all(chosen[clear] == best[clear])
    assert np.all(chosen <= best + 1e-4)


def test_nearest_level_at_the_thresholds():
    one = np.array([1.0], dtype=np.float32)
    # no-zero sets: exact midpoints go to the lower level; one ulp above goes up
    for lv, mids in ((oracle.MNZ, [-2.0, 0.0, 2.0]), (oracle.POT, [-2.5, 0.0, 2.5])):
        for i, m in enumerate(mids):
            m32 = np.float32(m)
            lo = np.nextafter(m32, np.float32(-np.inf))
            hi = np.nextafter(m32, np.float32(np.inf))
            w = np.array([[lo, m32, hi]], dtype=np.float32)
            assert oracle.assign_codes(w, lv, one)[0].tolist() == [i, i, i + 1]
        w = np.array([[-1e9, 1e9]], dtype=np.float32)
        assert oracle.assign_codes(w, lv, one)[0].tolist() == [0, 3]     # saturation
    # Eq. 1 sets: round half to even, then clip
    w = np.array([[-2.5, -1.5, -0.5, 0.5, 1.5, 9.0, -9.0]], dtype=np.float32)
    assert oracle.assign_codes(w, oracle.SYM, one)[0].tolist() == [0, 0, 2, 2, 3, 3, 0]
    w = np.array([[-8.5, -7.5, 6.5, 7.5, 100.0, -100.0, 0.0]], dtype=np.float32)
    q = [-8, -8, 6, 7, 7, -8, 0]
    assert oracle.assign_codes(w, oracle.INT4, one)[0].tolist() == [v & 15 for v in q]
    w = np.array([[-4.5, -3.5, -2.5, 2.5, 3.5, 0.5, 1.5, 50.0, -50.0, 0.0]], dtype=np.float32)
    q = [-4, -4, -2, 2, 3, 0, 2, 3, -4, 0]        # ties to even, then the clip to [-4, 3]
    assert oracle.assign_codes(w, oracle.INT3, one)[0].tolist() == [v & 7 for v in q]
    # a zero weight: MNZ/PoT code 1 (level -1), SYM code 2 (level 0), INT4 nibble 0
    z = np.zeros((1, 4), dtype=np.float32)
    assert oracle.assign_codes(z, oracle.MNZ, one)[0].tolist() == [1] * 4
    assert oracle.assign_codes(z, oracle.POT, one)[0].tolist() == [1] * 4
    assert oracle.assign_codes(z, oracle.SYM, one)[0].tolist() == [2] * 4
    assert oracle.assign_codes(z, oracle.INT4, one)[0].tolist() == [0] * 4


# ----------------------------------------------------------------------------- scale selection
def test_absmax_scale_and_zero_row():
    W = synth.gaussian_weights(0, 8, 64)
    W[3] = 0
    for lv, top in ((oracle.MNZ, 3), (oracle.POT, 4), (oracle.SYM, 1), (oracle.INT4, 7), (oracle.INT3, 3)):
        s, idx = oracle.weight_scale(W, lv, oracle.SCALE_ABSMAX)
        ref = np.abs(W).max(1) / np.float32(top)
        ref[3] = 1.0
        assert np.array_equal(s, ref.astype(np.float32))
        sm, _ = oracle.weight_scale(W, lv, oracle.SCALE_MSE)
        assert sm[3] == 1.0


def test_mse_sweep_definition():
    # candidates are the ratios 1.00, 0.99, ..., 0.21 and the winner is the first minimum of the
    # squared error recomputed here from nothing but the level table
    assert oracle.num_candidates() == 80
    assert [round(oracle.candidate_ratio(i), 2) for i in (0, 1, 79)] == [1.0, 0.99, 0.21]
    W = synth.gaussian_weights(5, 6, 512)
    for name, lv in list(LV.items()) + [("INT3", oracle.INT3)]:
        table = np.array(oracle.level_table(lv), dtype=np.float64)
        top = np.float32(table.max())
        s, idx, errs = oracle.weight_scale(W, lv, oracle.SCALE_MSE, want_errs=True)
        for n in range(W.shape[0]):
            amax = np.abs(W[n]).max()
            e_ref = []
            for i in range(80):
                p = np.float32(100 - i) / np.float32(100)
                si = np.float32(np.float32(p * amax) / top)
                w = W[n].astype(np.float64)
                rec = np.float64(si) * table[None, :]
                e_ref.append(((w[:, None] - rec) ** 2).min(1).sum())     # nearest level = least error
            e_ref = np.array(e_ref)
            assert np.allclose(errs[n], e_ref, rtol=1e-9)
            assert idx[n] == int(np.argmin(errs[n]))
            p = np.float32(100 - idx[n]) / np.float32(100)
            assert s[n] == np.float32(np.float32(p * amax) / top)


# ------------------------------------------------------------- Gaussian closed forms (Tables 13, 14)
def gaussian_quantizer_stats(levels, s):
    """Bucket probabilities and per-bucket squared error of nearest-level quantization of N(0,1)
    onto s*levels, by exact integrals."""
    L = np.array(levels, dtype=np.float64) * s
    edges = np.concatenate([[-np.inf], 0.5 * (L[1:] + L[:-1]), [np.inf]])
    a, b = edges[:-1], edges[1:]
    P = norm.cdf(b) - norm.cdf(a)
    with np.errstate(invalid="ignore"):
        pa = np.where(np.isinf(a), 0.0, a * norm.pdf(a))
        pb = np.where(np.isinf(b), 0.0, b * norm.pdf(b))
    m1 = norm.pdf(a) - norm.pdf(b)                      # int x phi
    m2 = P + pa - pb                                    # int x^2 phi
    err = m2 - 2 * L * m1 + L * L * P
    return P, err


def gaussian_optimum(levels):
    f = lambda s: gaussian_quantizer_stats(levels, s)[1].sum()
    res = optimize.minimize_scalar(f, bounds=(0.05, 3.0), method="bounded", options={"xatol": 1e-10})
    return res.x, res.fun


@pytest.fixture(scope="module")
def gaussian_rows():
    return synth.normal(77, 0, (256, 4096)).astype(np.float32)


def test_bucket_shares_reproduce_table13(gaussian_rows):
    W = gaussian_rows
    paper = {}
    rel = {}
    for row in read_golden("table13_buckets.txt"):
        if row[0] == "REL":
            rel[row[1]] = float(row[2])
        else:
            paper.setdefault(row[0], []).append((float(row[2]), float(row[3])))
    totals = {}
    for name, lv in LV.items():
        table = np.array(oracle.level_table(lv), dtype=np.float64)
        s, _ = oracle.weight_scale(W, lv, oracle.SCALE_MSE)
        codes = oracle.assign_codes(W, lv, s)
        rec = table[codes] * s[:, None].astype(np.float64)
        e = (W.astype(np.float64) - rec) ** 2
        cnt = np.array([(codes == c).mean() for c in range(4)]) * 100
        err = np.array([e[codes == c].sum() for c in range(4)]) / e.sum() * 100
        totals[name] = e.sum()
        # closed form at the Gaussian-optimal scale
        s_opt, _ = gaussian_optimum(table)
        P, E = gaussian_quantizer_stats(table, s_opt)
        assert np.abs(cnt - 100 * P).max() < 0.5, (name, cnt, 100 * P)
        assert np.abs(err - 100 * E / E.sum()).max() < 0.8, (name, err)
        # and the paper's measurement on real rotated weights
        pc = np.array([p[0] for p in paper[name]])
        pe = np.array([p[1] for p in paper[name]])
        assert np.abs(cnt - pc).max() < 0.6, (name, cnt, pc)
        assert np.abs(err - pe).max() < 1.0, (name, err, pe)
        # the scale the sweep finds is the Gaussian optimum (MNZ: Max's uniform 4-level step 0.9957)
        assert abs(np.median(s.astype(np.float64)) - s_opt) < 0.03 * s_opt
    for name in ("MNZ", "POT"):
        assert abs(totals[name] / totals["SYM"] - rel[name]) < 0.012
    assert totals["MNZ"] < totals["POT"] < totals["SYM"]


def test_best_scale_nmse_reproduces_table14(gaussian_rows):
    paper = {r[0]: (float(r[1]), float(r[2])) for r in read_golden("table14_ratio_nmse.txt")}
    x = gaussian_rows[:32].reshape(1, -1)                     # 131072 pooled samples
    power = (x.astype(np.float64) ** 2).sum()
    out = {}
    for name, lv, r in (("MNZ", oracle.MNZ, 1 / 3), ("POT", oracle.POT, 1 / 4)):
        top = oracle.level_table(lv)[3]
        _, closed = gaussian_optimum(np.array([-1, -r, r, 1.0]))
        s_opt, _ = gaussian_optimum(np.array(oracle.level_table(lv), dtype=np.float64))
        grid = np.float32(s_opt) * np.linspace(0.9, 1.1, 41, dtype=np.float32)
        nmse = min(oracle.row_sqerr(x[0], lv, float(s)) for s in grid) / power
        out[name] = nmse
        assert abs(nmse - closed) < 0.004 * closed + 1e-3          # sampling noise of 131K samples
        assert abs(nmse - paper[name][1]) < 0.02 * paper[name][1]
        assert abs(r - paper[name][0]) < 5e-5
    assert out["MNZ"] < out["POT"]                                 # same ordering as the table
    # closed forms alone reproduce the table's ordering, including the negative diagnostic r = 1/2
    closed = {k: gaussian_optimum(np.array([-1, -v[0], v[0], 1.0]))[1] for k, v in paper.items()}
    order = sorted(closed, key=closed.get)
    assert order.index("MNZ") < order.index("POT") < order.index("FAR")
    assert abs(closed["FAR"] - paper["FAR"][1]) < 0.01 * paper["FAR"][1]


def test_lloyd_max_levels_are_a_fixed_point():
    inner, outer = [float(v) for v in read_golden("lloyd_max_levels.txt")[0]]
    # Lloyd condition for N(0,1): each level is the centroid of its cell
    t = 0.5 * (inner + outer)
    c_in = (norm.pdf(0) - norm.pdf(t)) / (norm.cdf(t) - 0.5)
    c_out = norm.pdf(t) / (1 - norm.cdf(t))
    assert abs(c_in - inner) < 2e-4 and abs(c_out - outer) < 2e-4
    assert 0.25 < inner / outer < 1 / 3                        # the band that contains MNZ and PoT


# ----------------------------------------------------------------------------- packing (P8)
def tiled_address(n, j, words):
    """The storage order, written out independently of the oracle: 16-row x 128-word tiles, row
    blocks outermost; inside a tile 16-byte groups ordered (slice, half, row % 8, quad)."""
    pitch = -(-words // 16) * 16
    rb, r = divmod(n, 16)
    half, g = divmod(r, 8)
    c, jj = divmod(j, 128)
    sl, rem = divmod(jj, 16)
    quad, e = divmod(rem, 4)
    return rb * 16 * pitch + c * 2048 + (((sl * 2 + half) * 32 + g * 4 + quad) * 4 + e)


@pytest.mark.parametrize("lv", [oracle.MNZ, oracle.POT, oracle.SYM, oracle.INT4])
@pytest.mark.parametrize("N,words", [(5, 8), (16, 16), (37, 144), (33, 688)])
def test_pack_layout_and_roundtrip(lv, N, words):
    per, bits = (8, 4) if lv == oracle.INT4 else (16, 2)
    K = words * per
    rng = np.random.default_rng(3)
    pats = [rng.integers(0, 1 << bits, (N, K)), np.zeros((N, K)), np.full((N, K), (1 << bits) - 1),
            np.tile(np.arange(K) % (1 << bits), (N, 1))]
    n_pad, pitch = -(-N // 16) * 16, -(-words // 16) * 16
    # the address map is a bijection from (row, word) onto distinct slots of the padded buffer
    addr = np.array([[tiled_address(n, j, words) for j in range(words)] for n in range(N)])
    assert len(np.unique(addr)) == N * words and addr.max() < n_pad * pitch
    if words % 16 == 0 and N % 16 == 0:
        assert addr.max() == n_pad * pitch - 1
    for codes in pats:
        codes = codes.astype(np.uint8)
        p = oracle.pack(codes, lv)
        assert p.shape == (n_pad * pitch,) and p.dtype == np.uint32
        assert oracle.packed_words(N, K, lv) == n_pad * pitch
        assert np.array_equal(oracle.unpack(p, N, K, lv), codes)
        # bits inside a word: k = per*j + 4t + b -> bit 8b + bits*t
        ref = np.zeros((N, words), dtype=np.uint64)
        for k in range(K):
            j, r = divmod(k, per)
            t, b = divmod(r, 4)
            ref[:, j] |= codes[:, k].astype(np.uint64) << np.uint64(8 * b + bits * t)
        assert np.array_equal(p[addr], ref.astype(np.uint32))
        # padding slots are zero
        mask = np.ones(p.shape, dtype=bool)
        mask[addr.ravel()] = False
        assert not p[mask].any()
        # byte-lane property: (word >> bits*t) & mask gives four consecutive-k codes
        w = p[addr]
        m = 0x03030303 if bits == 2 else 0x0F0F0F0F
        for t in range(per // 4):
            lanes = ((w >> np.uint32(bits * t)) & np.uint32(m)).view(np.uint8).reshape(N, words, 4)
            want = codes.reshape(N, words, per // 4, 4)[:, :, t, :]
            assert np.array_equal(lanes, want)
    # a 16-byte group holds four consecutive words of one row; a warp's 32 groups are contiguous
    if words >= 16 and N >= 16:
        base = tiled_address(0, 0, words)
        for g in range(8):
            for quad in range(4):
                assert tiled_address(g, 4 * quad, words) == base + (g * 4 + quad) * 4
        assert tiled_address(8, 0, words) == base + 128          # rows 8..15: the next 512 bytes


def int3_addresses(n, j, pitch):
    """Low-plane and high-plane word of (row n, low word j), written from the layout's description: row blocks of
    24 * pitch words; slices of 16 low words = 384 words (256 low + 128 high)."""
    rb, r = divmod(n, 16)
    half, g = divmod(r, 8)
    sl, jj = divmod(j, 16)
    quad, e = divmod(jj, 4)
    base = rb * 24 * pitch + sl * 384
    return base + (half * 32 + g * 4 + quad) * 4 + e, base + 256 + (g * 4 + quad) * 4 + 2 * half + e // 2


@pytest.mark.parametrize("N,words", [(5, 8), (16, 16), (37, 144), (33, 688)])
def test_int3_plane_layout_and_roundtrip(N, words):
    K = words * 16
    rng = np.random.default_rng(4)
    n_pad, pitch = -(-N // 16) * 16, -(-words // 16) * 16
    total = n_pad * pitch * 3 // 2
    assert oracle.packed_words(N, K, oracle.INT3) == total
    lo = np.array([[int3_addresses(n, j, pitch)[0] for j in range(words)] for n in range(N)])
    hi = np.array([[int3_addresses(n, j, pitch)[1] for j in range(0, words, 2)] for n in range(N)])
    # both maps are injective, disjoint, inside the buffer; a pair of low words shares its high word
    allw = np.concatenate([lo.ravel(), hi.ravel()])
    assert len(np.unique(allw)) == allw.size and allw.max() < total
    assert all(int3_addresses(3, j, pitch)[1] == int3_addresses(3, j + 1, pitch)[1] for j in range(0, words, 2))
    pats = [rng.integers(0, 8, (N, K)), np.zeros((N, K)), np.full((N, K), 7), np.tile(np.arange(K) % 8, (N, 1)),
            np.full((N, K), 4), np.full((N, K), 3)]
    for codes in pats:
        codes = codes.astype(np.uint8)
        p = oracle.pack(codes, oracle.INT3)
        assert p.shape == (total,)
        assert np.array_equal(oracle.unpack(p, N, K, oracle.INT3), codes)
        # low plane: exactly the two-bit word of the codes' low bits
        ref_lo = np.zeros((N, words), dtype=np.uint64)
        ref_hi = np.zeros((N, words // 2), dtype=np.uint64)
        for k in range(K):
            j, r = divmod(k, 16)
            t, b = divmod(r, 4)
            ref_lo[:, j] |= (codes[:, k] & 3).astype(np.uint64) << np.uint64(8 * b + 2 * t)
            ref_hi[:, j // 2] |= (codes[:, k] >> 2).astype(np.uint64) << np.uint64(8 * b + 4 * (j % 2) + (0, 2, 1, 3)[t])
        assert np.array_equal(p[lo], ref_lo.astype(np.uint32))
        assert np.array_equal(p[hi], ref_hi.astype(np.uint32))
        mask = np.ones(p.shape, dtype=bool)
        mask[allw] = False
        assert not p[mask].any()
    # the property the storage is built for: in a high word, the bits of planes t and t + 1 of a low word lie
    # two positions apart (t even), so that with the even planes' activations scaled by four both halves of a
    # product step carry the same place value
    for par in range(2):
        for t in (0, 2):
            b0 = 4 * par + (0, 2, 1, 3)[t]
            b1 = 4 * par + (0, 2, 1, 3)[t + 1]
            assert b1 == b0 + 2
    # three bits per weight on the paper's shapes, no padding
    for _, n, k in synth.LLAMA2_7B + synth.LLAMA31_8B:
        assert oracle.packed_words(n, k, oracle.INT3) * 32 == 3 * n * k
    # a slice of a row block is contiguous: 16 rows x 16 low words and their high words in 384 words
    a = sorted([int3_addresses(n, j, 16)[0] for n in range(16) for j in range(16)] +
               list({int3_addresses(n, j, 16)[1] for n in range(16) for j in range(16)}))
    assert a == list(range(384))


def test_packed_bytes_of_llama_shapes():
    # no padding on the paper's shapes: exactly 2 (or 4) bits per weight
    for _, N, K in synth.LLAMA2_7B + synth.LLAMA31_8B:
        assert oracle.packed_words(N, K, oracle.MNZ) * 4 == N * K // 4
        assert oracle.packed_words(N, K, oracle.INT4) * 4 == N * K // 2


def test_mixed_stack_is_three_bits_per_weight():
    # L = 16 of 32 layers at 4 bits, the rest at 2: b_avg = 2 + L/16 = 3 (Sec. 4.4)
    per_layer = sum(n * k for _, n, k in synth.LLAMA2_7B)
    bits = 16 * per_layer * 4 + 16 * per_layer * 2
    assert bits / (32 * per_layer) == 3.0 == 2 + 16 / 16


# ----------------------------------------------------------------------------- integer product (P11)
@pytest.mark.parametrize("name", ["MNZ", "POT", "SYM"])
def test_product_exhaustive_k4(name):
    lv = LV[name]
    key = {"MNZ": "MNZ_INT", "POT": "POT", "SYM": "SYM"}[name]
    table = np.array(paper_levels()[key], dtype=np.int64)            # the paper's levels, not the oracle's
    codes = np.array(list(itertools.product(range(4), repeat=4)), dtype=np.uint8)          # 256 x 4
    acts = np.array(list(itertools.product(range(-8, 8), repeat=4)), dtype=np.int8)        # 65536 x 4
    acc = oracle.int_matmul(codes, lv, acts)
    ref = acts.astype(np.int64) @ table[codes].T
    assert np.array_equal(acc.astype(np.int64), ref)


def test_product_exhaustive_int3_k3():
    # Eq. 1 with b = 3: the decoded level of the two's-complement field c is c - 8 [c >= 4]
    table = np.array([c - 8 if c >= 4 else c for c in range(8)], dtype=np.int64)
    codes = np.array(list(itertools.product(range(8), repeat=3)), dtype=np.uint8)           # 512 x 3
    acts = np.array(list(itertools.product(range(-8, 8), repeat=3)), dtype=np.int8)         # 4096 x 3
    acc = oracle.int_matmul(codes, oracle.INT3, acts)
    assert np.array_equal(acc.astype(np.int64), acts.astype(np.int64) @ table[codes].T)


def test_product_closed_cases_and_library_crosscheck():
    import torch
    rng = np.random.default_rng(8)
    M, N, K = 3, 7, 160
    q = rng.integers(-8, 8, (M, K)).astype(np.int8)
    for lv in (oracle.MNZ, oracle.POT, oracle.SYM, oracle.INT4, oracle.INT3):
        nc = oracle.num_codes(lv)
        table = np.array(oracle.level_table(lv), dtype=np.int64)
        codes = rng.integers(0, nc, (N, K)).astype(np.uint8)
        acc = oracle.int_matmul(codes, lv, q)
        ref = torch.from_numpy(q.astype(np.int64)) @ torch.from_numpy(table[codes]).T
        assert np.array_equal(acc, ref.numpy().astype(np.int32))
        assert np.abs(acc).max() <= K * np.abs(table).max() * 8
        assert not oracle.int_matmul(codes, lv, np.zeros_like(q)).any()
        if lv in (oracle.MNZ, oracle.POT):      # mirrored codes negate the product
            assert np.array_equal(oracle.int_matmul(3 - codes, lv, q), -acc)
        if lv == oracle.INT3:                   # plane form: low two bits minus four times the third
            q64 = q.astype(np.int64)
            assert np.array_equal(acc, q64 @ (codes & 3).astype(np.int64).T - 4 * (q64 @ (codes >> 2).astype(np.int64).T))
        elif lv != oracle.INT4:                 # bit-plane form as a second formula
            a, b, c = {oracle.MNZ: (4, 2, -3), oracle.POT: (5, 3, -4), oracle.SYM: (2, 1, -2)}[lv]
            b1, b0 = (codes >> 1).astype(np.int64), (codes & 1).astype(np.int64)
            q64 = q.astype(np.int64)
            alt = a * (q64 @ b1.T) + b * (q64 @ b0.T) + c * q64.sum(1, keepdims=True)
            assert np.array_equal(acc, alt)
    top = np.full((2, 64), 3, dtype=np.uint8)
    assert np.all(oracle.int_matmul(top, oracle.MNZ, np.full((1, 64), 7, dtype=np.int8)) == 21 * 64)
    # largest accumulator of any configured shape stays exactly representable in fp32
    assert 14336 * 8 * 8 < 2 ** 24


# ----------------------------------------------------------------------------- epilogue (P12)
def test_epilogue_order_and_rounding():
    import torch
    rng = np.random.default_rng(2)
    M, N = 4, 300
    acc = rng.integers(-917504, 917505, (M, N)).astype(np.int32)
    s_a = (rng.random(M) * 0.3 + 0.01).astype(np.float32)
    s_n = (rng.random(N) * 0.01 + 1e-4).astype(np.float32)
    y = oracle.epilogue(acc, s_a, s_n)
    # pinned multiply order (acc * s_a) * s_n, each a single fp32 operation
    ref = (acc.astype(np.float32) * s_a[:, None]) * s_n[None, :]
    assert np.array_equal(y, ref)
    exact = acc.astype(np.float64) * s_a[:, None].astype(np.float64) * s_n[None, :].astype(np.float64)
    assert np.all(np.abs(y - exact) <= 2 * np.spacing(np.abs(y)))
    yb = oracle.epilogue(acc, s_a, s_n, bf16=True)
    refb = torch.from_numpy(ref).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(yb, refb)


def test_whole_layer_on_config1_matches_the_dequantized_definition():
    # y = s_n * sum_k level * q_a * s_a, evaluated in fp64 from the decoded quantities
    W = synth.gaussian_weights(0, 256, 256)
    x, _ = synth.activations(1, 1, 256, 4)
    packed, s_n, codes = oracle.pack_weights(W, oracle.MNZ, oracle.SCALE_MSE)
    q_a, s_a = oracle.quantize_act(x, 256, 0.9)
    y, acc = oracle.linear(oracle.unpack(packed, 256, 256, oracle.MNZ), oracle.MNZ, s_n, q_a, s_a)
    table = np.array(paper_levels()["MNZ_INT"])
    w_hat = table[codes] * s_n[:, None].astype(np.float64)
    a_hat = q_a.astype(np.float64) * s_a[:, None].astype(np.float64)
    ref = a_hat @ w_hat.T
    assert np.allclose(y, ref, rtol=1e-5, atol=1e-9)
    # and the quantized layer approximates the fp layer on the rotated operands
    full = oracle.rotate_weights(x, 256).astype(np.float64) @ W.astype(np.float64).T
    rel = np.linalg.norm(y - full) / np.linalg.norm(full)
    assert rel < 0.6

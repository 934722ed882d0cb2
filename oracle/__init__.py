"""CPU oracle for the Qift quantized linear layer -- TEST INFRASTRUCTURE ONLY.

A ctypes front end to ``qift_oracle.cpp`` (plain single-threaded C++17, compiled with
``g++ -O2 -ffp-contract=off``).  The oracle restates what the paper's layer computes; it shares no
code with the CUDA library and must never be imported by it.  Only tests, the smoke check and the
CPU-baseline / reference legs of the benchmark may use this package.

All arrays are numpy, C-contiguous.  Level-set ids: 0 MNZ {-3,-1,+1,+3} (half-scale form of
{+-0.5,+-1.5}), 1 PoT-MNZ {-4,-1,+1,+4}, 2 SYM-INT {-2,-1,0,+1}, 3 INT4 (-8..7), 4 INT3 (-4..3, the W3A4
configuration of Sec. 4.4).
Scale modes: 0 given, 1 max-range, 2 MSE sweep over 80 clipping ratios.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

MNZ, POT, SYM, INT4, INT3 = 0, 1, 2, 3, 4
SCALE_GIVEN, SCALE_ABSMAX, SCALE_MSE = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qift_oracle.cpp")
_LIB = os.path.join(_HERE, "libqift_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle shared library beside its source (no-op when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC", _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, t):
    return a.ctypes.data_as(ctypes.POINTER(t))


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_candidate_ratio.restype = ctypes.c_float
        _lib.orc_row_sqerr.restype = ctypes.c_double
        _lib.orc_row_sqerr.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_float]
        _lib.orc_int_matmul.restype = ctypes.c_longlong
        _lib.orc_packed_words.restype = ctypes.c_longlong
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def level_value(lv: int, code: int) -> int:
    return int(lib().orc_level_value(int(lv), int(code)))


def num_codes(lv: int) -> int:
    return 16 if lv == INT4 else 8 if lv == INT3 else 4


def level_table(lv: int):
    return [level_value(lv, c) for c in range(num_codes(lv))]


def num_candidates() -> int:
    return int(lib().orc_num_candidates())


def candidate_ratio(i: int) -> float:
    return float(lib().orc_candidate_ratio(int(i)))


def wht_blocks(x, B: int):
    """Unnormalised blockwise Walsh-Hadamard transform of each row (fp32 butterfly)."""
    x = _f32(x).copy()
    rows = x.reshape(-1, x.shape[-1])
    K = rows.shape[1]
    assert B >= 1 and (B & (B - 1)) == 0 and K % B == 0
    for r in rows:
        lib().orc_wht_blocks(r.ctypes.data_as(ctypes.c_void_p), K, B)
    return x


def is_kron28(K: int, B: int) -> bool:
    """B == K == 28 * 2^p selects the full-dimension rotation H_28 (x) H_{2^p}."""
    P = K // 28
    return B == K and K % 28 == 0 and P >= 1 and (P & (P - 1)) == 0


def hadamard28():
    H = np.empty((28, 28), dtype=np.int8)
    lib().orc_hadamard28(H.ctypes.data_as(ctypes.c_void_p))
    return H


def rotate_weights(W, B: int):
    """W Q with Q = blockdiag(H_B)/sqrt(B) along the last axis (fp32); B = K = 28 * 2^p: full-dimension rotation."""
    W = _f32(W).copy()
    N, K = W.shape
    assert ((B & (B - 1)) == 0 and K % B == 0) or is_kron28(K, B)
    lib().orc_rotate_weights(W.ctypes.data_as(ctypes.c_void_p), N, K, B)
    return W


def bf16_to_f32(u16):
    u16 = np.ascontiguousarray(u16, dtype=np.uint16)
    out = np.empty(u16.shape, dtype=np.float32)
    lib().orc_bf16_to_f32(u16.ctypes.data_as(ctypes.c_void_p), out.ctypes.data_as(ctypes.c_void_p),
                          ctypes.c_longlong(u16.size))
    return out


def f32_to_bf16(x):
    x = _f32(x)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().orc_f32_to_bf16(x.ctypes.data_as(ctypes.c_void_p), out.ctypes.data_as(ctypes.c_void_p),
                          ctypes.c_longlong(x.size))
    return out


def quantize_act(X, had_block: int, clip: float = 0.9):
    """-> (q_a int8 [M,K], s_a fp32 [M])."""
    X = _f32(X)
    M, K = X.shape
    assert had_block == 0 or ((had_block & (had_block - 1)) == 0 and K % had_block == 0) or is_kron28(K, had_block)
    q = np.empty((M, K), dtype=np.int8)
    s = np.empty((M,), dtype=np.float32)
    scratch = np.empty((K,), dtype=np.float32)
    lib().orc_quantize_act(X.ctypes.data_as(ctypes.c_void_p), M, K, int(had_block),
                           ctypes.c_float(clip), q.ctypes.data_as(ctypes.c_void_p),
                           s.ctypes.data_as(ctypes.c_void_p), scratch.ctypes.data_as(ctypes.c_void_p))
    return q, s


def row_sqerr(w, lv: int, s: float) -> float:
    w = _f32(w)
    return float(lib().orc_row_sqerr(w.ctypes.data_as(ctypes.c_void_p), w.size, int(lv),
                                     ctypes.c_float(s)))


def weight_scale(W, lv: int, mode: int, want_errs: bool = False):
    """-> (s_n fp32 [N], best_idx int32 [N][, errs fp64 [N,80]])."""
    W = _f32(W)
    N, K = W.shape
    s = np.empty((N,), dtype=np.float32)
    idx = np.zeros((N,), dtype=np.int32)
    errs = np.zeros((N, num_candidates()), dtype=np.float64) if want_errs else None
    lib().orc_weight_scale(W.ctypes.data_as(ctypes.c_void_p), N, K, int(lv), int(mode),
                           s.ctypes.data_as(ctypes.c_void_p), idx.ctypes.data_as(ctypes.c_void_p),
                           errs.ctypes.data_as(ctypes.c_void_p) if want_errs else None)
    return (s, idx, errs) if want_errs else (s, idx)


def assign_codes(W, lv: int, s_n):
    W = _f32(W)
    s_n = _f32(s_n)
    N, K = W.shape
    codes = np.empty((N, K), dtype=np.uint8)
    lib().orc_assign_codes(W.ctypes.data_as(ctypes.c_void_p), N, K, int(lv),
                           s_n.ctypes.data_as(ctypes.c_void_p), codes.ctypes.data_as(ctypes.c_void_p))
    return codes


def codes_per_word(lv: int) -> int:
    """Codes per 32-bit word (INT3: of its two-bit plane; K must then be a multiple of 32)."""
    return 8 if lv == INT4 else 16


def packed_words(N: int, K: int, lv: int) -> int:
    """Words of the packed buffer: rows padded to a multiple of 16."""
    return int(lib().orc_packed_words(N, K, int(lv)))


def pack(codes, lv: int):
    """codes uint8 [N,K] -> flat uint32 buffer in the tiled layout."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape
    per = 32 if lv == INT3 else codes_per_word(lv)
    assert K % per == 0
    out = np.empty((packed_words(N, K, lv),), dtype=np.uint32)
    lib().orc_pack(codes.ctypes.data_as(ctypes.c_void_p), N, K, int(lv),
                   out.ctypes.data_as(ctypes.c_void_p))
    return out


def unpack(packed, N: int, K: int, lv: int):
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    assert packed.size == packed_words(N, K, lv)
    out = np.empty((N, K), dtype=np.uint8)
    lib().orc_unpack(packed.ctypes.data_as(ctypes.c_void_p), N, K, int(lv),
                     out.ctypes.data_as(ctypes.c_void_p))
    return out


def int_matmul(codes, lv: int, q_a):
    """acc int32 [M,N] = sum_k level(code[n,k]) * q_a[m,k]; asserts no int32 overflow."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    q_a = np.ascontiguousarray(q_a, dtype=np.int8)
    N, K = codes.shape
    M, K2 = q_a.shape
    assert K == K2
    acc = np.empty((M, N), dtype=np.int32)
    bad = lib().orc_int_matmul(codes.ctypes.data_as(ctypes.c_void_p), int(lv),
                               q_a.ctypes.data_as(ctypes.c_void_p), M, N, K,
                               acc.ctypes.data_as(ctypes.c_void_p))
    assert bad == 0, "int32 accumulator overflow"
    return acc


def epilogue(acc, s_a, s_n, bf16: bool = False):
    """y = ((float)acc * s_a[m]) * s_n[n]; fp32, or bf16 bit patterns (uint16) by RNE."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    s_a = _f32(s_a)
    s_n = _f32(s_n)
    M, N = acc.shape
    if bf16:
        y = np.empty((M, N), dtype=np.uint16)
        fn = lib().orc_epilogue_bf16
    else:
        y = np.empty((M, N), dtype=np.float32)
        fn = lib().orc_epilogue
    fn(acc.ctypes.data_as(ctypes.c_void_p), s_a.ctypes.data_as(ctypes.c_void_p),
       s_n.ctypes.data_as(ctypes.c_void_p), M, N, y.ctypes.data_as(ctypes.c_void_p))
    return y


def pack_weights(W, lv: int, mode: int, s_n=None):
    """Whole S1 step -> (packed uint32 flat (tiled layout), s_n, codes)."""
    if mode == SCALE_GIVEN:
        s = _f32(s_n)
    else:
        s, _ = weight_scale(W, lv, mode)
    codes = assign_codes(W, lv, s)
    return pack(codes, lv), s, codes


def linear(codes, lv: int, s_n, q_a, s_a, bf16: bool = False):
    """S4 + S5 -> (y, acc)."""
    acc = int_matmul(codes, lv, q_a)
    return epilogue(acc, s_a, s_n, bf16=bf16), acc


# ---------------------------------------------------------------------------------------- KV4
def kv4_quantize(X, had_block: int = 0, clip: float = 0.95):
    """X fp32 [rows, D] -> (codes uint8 [rows, D] in 0..15, scale fp32 [rows], zero fp32 [rows])."""
    X = _f32(X)
    rows, D = X.shape
    assert had_block == 0 or ((had_block & (had_block - 1)) == 0 and D % had_block == 0)
    codes = np.empty((rows, D), dtype=np.uint8)
    scale = np.empty((rows,), dtype=np.float32)
    zero = np.empty((rows,), dtype=np.float32)
    scratch = np.empty((D,), dtype=np.float32)
    vp = ctypes.c_void_p
    lib().orc_kv4_quantize(X.ctypes.data_as(vp), ctypes.c_longlong(rows), D, int(had_block), ctypes.c_float(clip),
                           codes.ctypes.data_as(vp), scale.ctypes.data_as(vp), zero.ctypes.data_as(vp),
                           scratch.ctypes.data_as(vp))
    return codes, scale, zero


def kv4_pack(codes):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    rows, D = codes.reshape(-1, codes.shape[-1]).shape
    out = np.empty((rows, D // 2), dtype=np.uint8)
    vp = ctypes.c_void_p
    lib().orc_kv4_pack(codes.ctypes.data_as(vp), ctypes.c_longlong(rows), D, out.ctypes.data_as(vp))
    return out.reshape(codes.shape[:-1] + (D // 2,))


def kv4_pack_token_pairs(codes):
    """codes uint8 [H, T, D] (T even) -> bytes uint8 [H, T/2, D]: tokens 2i (low nibble) and 2i+1 of a dimension per byte."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    H, T, D = codes.shape
    assert T % 2 == 0
    out = np.empty((H, T // 2, D), dtype=np.uint8)
    vp = ctypes.c_void_p
    for h in range(H):
        lib().orc_kv4_pack_token_pairs(codes[h].ctypes.data_as(vp), ctypes.c_longlong(T), D, out[h].ctypes.data_as(vp))
    return out


def kv4_unpack(packed):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    rows, half = packed.reshape(-1, packed.shape[-1]).shape
    out = np.empty((rows, 2 * half), dtype=np.uint8)
    vp = ctypes.c_void_p
    lib().orc_kv4_unpack(packed.ctypes.data_as(vp), ctypes.c_longlong(rows), 2 * half, out.ctypes.data_as(vp))
    return out.reshape(packed.shape[:-1] + (2 * half,))


def kv4_attention(q, kc, ks, kz, vc, vs, vz):
    """q fp32 [Hq, D]; codes uint8 [Hkv, T, D]; scales / zero-points fp32 [Hkv, T] -> out fp64 [Hq, D]."""
    q = _f32(q)
    Hq, D = q.shape
    kc = np.ascontiguousarray(kc, dtype=np.uint8)
    vc = np.ascontiguousarray(vc, dtype=np.uint8)
    Hkv, T, D2 = kc.shape
    assert D2 == D and vc.shape == kc.shape and Hq % Hkv == 0
    ks, kz, vs, vz = (_f32(a) for a in (ks, kz, vs, vz))
    out = np.empty((Hq, D), dtype=np.float64)
    scratch = np.empty((T,), dtype=np.float64)
    vp = ctypes.c_void_p
    lib().orc_kv4_attention(q.ctypes.data_as(vp), kc.ctypes.data_as(vp), ks.ctypes.data_as(vp), kz.ctypes.data_as(vp),
                            vc.ctypes.data_as(vp), vs.ctypes.data_as(vp), vz.ctypes.data_as(vp), T, Hq, Hkv, D,
                            out.ctypes.data_as(vp), scratch.ctypes.data_as(vp))
    return out


# ------------------------------------------------------------------ quantizer diagnostics (Sec. 4.5)
def _grid(g):
    g = _f32(g).reshape(-1)
    assert g.size == 4 and np.all(np.diff(g) > 0) and g[3] > 0
    return g


def grid_scale(W, grid, mode: int, want_errs: bool = False):
    """Per-row scale of a four-level float grid -> (s_n fp32 [N], best_idx int32 [N][, errs fp64 [N,80]])."""
    W = _f32(W)
    g = _grid(grid)
    N, K = W.shape
    s = np.empty((N,), dtype=np.float32)
    idx = np.zeros((N,), dtype=np.int32)
    errs = np.zeros((N, num_candidates()), dtype=np.float64) if want_errs else None
    vp = ctypes.c_void_p
    lib().orc_grid_scale(W.ctypes.data_as(vp), N, K, g.ctypes.data_as(vp), int(mode), s.ctypes.data_as(vp),
                         idx.ctypes.data_as(vp), errs.ctypes.data_as(vp) if want_errs else None)
    return (s, idx, errs) if want_errs else (s, idx)


def grid_codes(W, grid, s_n):
    W = _f32(W)
    g = _grid(grid)
    s_n = _f32(s_n)
    N, K = W.shape
    codes = np.empty((N, K), dtype=np.uint8)
    vp = ctypes.c_void_p
    lib().orc_grid_codes(W.ctypes.data_as(vp), N, K, g.ctypes.data_as(vp), s_n.ctypes.data_as(vp),
                         codes.ctypes.data_as(vp))
    return codes


def bucket_stats(W, codes, s_n, values):
    """-> (count int64 [L], sqerr fp64 [L]) of the weights assigned to each of the L levels."""
    W = _f32(W)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    s_n = _f32(s_n)
    v = _f32(values).reshape(-1)
    N, K = W.shape
    assert codes.shape == W.shape and int(codes.max(initial=0)) < v.size
    count = np.zeros((v.size,), dtype=np.int64)
    sqerr = np.zeros((v.size,), dtype=np.float64)
    vp = ctypes.c_void_p
    lib().orc_bucket_stats(W.ctypes.data_as(vp), codes.ctypes.data_as(vp), N, K, s_n.ctypes.data_as(vp),
                           v.ctypes.data_as(vp), v.size, count.ctypes.data_as(vp), sqerr.ctypes.data_as(vp))
    return count, sqerr


def ratio_scan(x, ratios):
    """-> (beta fp64 [R], nmse fp64 [R]): best global scale and its NMSE for each grid {-1,-r,+r,+1}."""
    x = _f32(x).reshape(-1)
    r = np.ascontiguousarray(ratios, dtype=np.float64).reshape(-1)
    beta = np.empty_like(r)
    nmse = np.empty_like(r)
    vp = ctypes.c_void_p
    lib().orc_ratio_scan(x.ctypes.data_as(vp), ctypes.c_longlong(x.size), r.ctypes.data_as(vp), r.size,
                         beta.ctypes.data_as(vp), nmse.ctypes.data_as(vp))
    return beta, nmse

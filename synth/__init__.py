"""Seeded synthetic inputs shared by the oracle-side and the CUDA-side of every parity test.

Nothing here is part of the quantization method: this module only draws numbers.  It stands in for
the LLaMA-2-7B / LLaMA-3.1-8B weights and the WikiText-2 activations the paper measures on (neither
is available offline): same shapes, zero-mean Gaussian or heavy-tailed Student-t(5) weights (the
paper's pre-rotation weights have excess kurtosis of a few units, Table 3), Gaussian activations
with a small set of outlier channels (Figure 1).

Generator: counter-based.  element i of tensor (seed, tensor_id) takes two 64-bit words
splitmix64(key + 2i), splitmix64(key + 2i + 1) -> two uniforms in (0,1) -> one variate, all in
fp64, cast to fp32 at the end.  Any slice of a tensor can therefore be drawn on its own.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)

# (name, N, K) of the seven linear modules of one transformer layer.
LLAMA2_7B = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
             ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
LLAMA31_8B = [("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
              ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336)]


def had_block_for(K: int) -> int:
    """Largest power of two dividing K (the block size of the block-diagonal rotation)."""
    return K & (-K)


def _splitmix64(x):
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = x
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int) -> np.uint64:
    k = _splitmix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    k = _splitmix64(k ^ np.uint64(tensor_id & 0xFFFFFFFF))
    return k[0]


def uniforms(seed: int, tensor_id: int, n: int, offset: int = 0):
    """Two independent fp64 uniforms in (0,1) for each of n elements starting at `offset`."""
    key = _key(seed, tensor_id)
    idx = (np.arange(n, dtype=np.uint64) + np.uint64(offset)) * np.uint64(2)
    with np.errstate(over="ignore"):
        a = _splitmix64(key + idx)
        b = _splitmix64(key + idx + np.uint64(1))
    scale = 1.0 / 9007199254740992.0  # 2^-53
    u = ((a >> np.uint64(11)).astype(np.float64) + 0.5) * scale
    v = ((b >> np.uint64(11)).astype(np.float64) + 0.5) * scale
    return u, v


_CHUNK = 1 << 18   # elements drawn per task: the temporaries of a task stay in cache


def _draw(variate, seed: int, tensor_id: int, shape, offset: int):
    """Fills an fp64 array element by element from the counter-based stream.  Element i depends on
    (seed, tensor_id, offset + i) only, so the array is cut into chunks that worker threads draw
    independently (numpy releases the interpreter lock inside its loops); the values do not depend
    on the chunking."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float64)

    def task(lo):
        hi = min(n, lo + _CHUNK)
        u, v = uniforms(seed, tensor_id, hi - lo, offset + lo)
        out[lo:hi] = variate(u, v)

    starts = range(0, n, _CHUNK)
    if n <= _CHUNK:
        for lo in starts:
            task(lo)
    else:
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
            list(pool.map(task, starts))
    return out.reshape(shape)


def normal(seed: int, tensor_id: int, shape, offset: int = 0):
    """iid N(0,1), fp64 (Box-Muller cosine branch)."""
    return _draw(lambda u, v: np.sqrt(-2.0 * np.log(u)) * np.cos(2.0 * np.pi * v), seed, tensor_id, shape, offset)


def student_t(seed: int, tensor_id: int, shape, df: float = 5.0, offset: int = 0):
    """iid Student-t(df), fp64 (Bailey's polar form: sqrt(df (u^(-2/df) - 1)) cos(2 pi v))."""
    return _draw(lambda u, v: np.sqrt(df * (np.power(u, -2.0 / df) - 1.0)) * np.cos(2.0 * np.pi * v), seed, tensor_id,
                 shape, offset)


def choose_channels(seed: int, tensor_id: int, K: int, count: int):
    """`count` distinct channel indices in [0, K), sorted (rank of per-channel uniforms)."""
    u, _ = uniforms(seed, tensor_id, K)
    return np.sort(np.argsort(u, kind="stable")[:count])


def gaussian_weights(seed: int, N: int, K: int, sigma: float = 0.02, tensor_id: int = 0):
    """W ~ N(0, sigma^2) iid, fp32 [N, K]."""
    return (sigma * normal(seed, tensor_id, (N, K))).astype(np.float32)


def student_weights(seed: int, N: int, K: int, sigma: float = 0.02, df: float = 5.0,
                    tensor_id: int = 0):
    """W = sigma * t_df iid, fp32 [N, K] (heavy-tailed stand-in for un-rotated weights)."""
    return (sigma * student_t(seed, tensor_id, (N, K), df)).astype(np.float32)


def activations(seed: int, M: int, K: int, n_outliers: int, mult: float = 20.0, tensor_id: int = 1):
    """x ~ N(0,1) fp32 [M, K]; a fixed seeded set of `n_outliers` channels is multiplied by `mult`
    in every row.  Returns (x, outlier_channel_indices)."""
    x = normal(seed, tensor_id, (M, K))
    ch = choose_channels(seed, tensor_id + 1, K, n_outliers)
    x[:, ch] *= mult
    return x.astype(np.float32), ch


def config_seed(config: int, shape_idx: int, what: int) -> int:
    """Seed convention: 1000*config + 10*shape + {0 weights, 1 activations}."""
    return 1000 * config + 10 * shape_idx + what

// K2, second form: rotate + quantize one token row per CTA with every element living in ONE thread's
// registers between passes -- 32 elements per thread, K / 32 threads per row.
//
// The transform of a block of B = 2^b entries is b butterfly stages in ascending stride.  They are cut into at
// most three passes; inside a pass a thread owns all partners of its elements, so the stages of a pass run in
// registers, and the row crosses shared memory only between passes (padded layout of rotate_quant.cuh):
//   first pass    32 contiguous elements straight from global memory: strides 1 .. 16 (stride 1 on scalars,
//                 then packed fp32 pairs of neighbours)
//   middle pass   only when more than four stages are left: strides 32 .. 256 on 16 rows x 2 neighbouring
//                 columns, in place
//   last pass     the remaining r <= 4 stages on 2^r rows x 32 / 2^r neighbouring columns.  The thread keeps
//                 its 32 values in registers across the row-maximum reduction and quantizes them from there:
//                 no write-back of the transformed row, no second read.
// Every stage is the same set of independent IEEE additions as the in-place butterfly, so the result is
// bit-identical to it; the row maximum is order-independent; the quantizer is the division-free one of
// rotate_quant.cuh (reciprocal multiply, exact quotient for any group with an element near a rounding tie).
// Serves power-of-two blocks up to 8192 (and no rotation) for K a multiple of 32; the general kernel
// (quantize_act_kernel) keeps B = 16384, K not a multiple of 32 and the 28-point Kronecker factor.
#pragma once

#include "common.cuh"
#include "rotate_quant.cuh"

namespace qift {

constexpr int kRowsMaxThreads = 512;  // K <= 16384

__device__ __forceinline__ float fmax3_abs(float m, float a, float b) { return fmaxf(m, fmaxf(fabsf(a), fabsf(b))); }

// Row scale from the threads' partial maxima with ONE barrier: every warp leaves its maximum in shared memory,
// and after the barrier every thread reduces the (at most 16) warp maxima itself and derives s_u and 1 / s_u
// (the same few operations in every thread, instead of a second barrier to broadcast them).  `red` alternates
// between two sets of 16 slots from row to row, so a warp that is already at the next row's reduction cannot
// overwrite maxima that a slower warp has not read yet.
__device__ __forceinline__ RowScale block_row_scale_wide(float v, float clip, float* red, int parity) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    float* slot = red + 16 * parity;
    if (lane == 0) slot[warp] = v;
    __syncthreads();
    float r = 0.0f;
    for (int w = 0; w < warps; w += 4) {
        const float4 f = *reinterpret_cast<const float4*>(slot + w);
        r = fmaxf(fmaxf(r, f.x), fmaxf(w + 1 < warps ? f.y : 0.0f, fmaxf(w + 2 < warps ? f.z : 0.0f, w + 3 < warps ? f.w : 0.0f)));
    }
    float s_u = 1.0f;
    if (r != 0.0f) s_u = __fdiv_rn(__fmul_rn(r, clip), 7.0f);
    const bool fast = (s_u >= 1e-30f) && (s_u <= 1e30f);
    return RowScale{s_u, fast ? __fdiv_rn(1.0f, s_u) : 0.0f};
}

// Fast quantization of NP pairs (2 NP neighbouring elements) held in registers: y[i] = clamp(u * (1 / s_u)) +
// 1.5 * 2^23, whose low byte per half is the rounded integer.  Adds to `dmax` the largest distance of a clamped
// quotient from its rounded value: above kTieGuard the caller redoes its elements with exact quotients.
// UPPER_ONLY: |u| * (1 / s_u) stays below 8.5, so only the clamp at +7 can act.
template <int NP, bool UPPER_ONLY>
__device__ __forceinline__ void quantize_pairs_fast(const f32x2_t (&u)[NP], f32x2_t inv2, f32x2_t (&y)[NP], float& dmax) {
    const f32x2_t magic2 = f2_make(kRoundMagic, kRoundMagic);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        float t0, t1;
        f2_split(f2_mul(u[i], inv2), t0, t1);
        if (UPPER_ONLY) t0 = fminf(t0, 7.0f), t1 = fminf(t1, 7.0f);
        else t0 = fminf(fmaxf(t0, -8.0f), 7.0f), t1 = fminf(fmaxf(t1, -8.0f), 7.0f);
        const f32x2_t t2 = f2_make(t0, t1);
        y[i] = f2_add(t2, magic2);
        float d0, d1;
        f2_split(f2_sub(t2, f2_sub(y[i], magic2)), d0, d1);
        dmax = fmax3_abs(dmax, d0, d1);
    }
}
template <int NP>
__device__ __forceinline__ void quantize_pairs_exact(const f32x2_t (&u)[NP], float s_u, f32x2_t (&y)[NP]) {
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        float u0, u1;
        f2_split(u[i], u0, u1);
        y[i] = f2_make(__fadd_rn(quantize_round_exact(u0, s_u), kRoundMagic), __fadd_rn(quantize_round_exact(u1, s_u), kRoundMagic));
    }
}
// The low bytes of the 2 NP halves, four per word (NP = 1: the low half word of out[0]).
template <int NP>
__device__ __forceinline__ void low_bytes(const f32x2_t (&y)[NP], uint32_t (&out)[(NP + 1) / 2]) {
#pragma unroll
    for (int i = 0; i < (NP + 1) / 2; ++i) {
        float b0, b1, b2 = 0.0f, b3 = 0.0f;
        f2_split(y[2 * i], b0, b1);
        if (2 * i + 1 < NP) f2_split(y[2 * i + 1], b2, b3);
        out[i] = __byte_perm(__byte_perm(__float_as_uint(b0), __float_as_uint(b1), 0x0040),
                             __byte_perm(__float_as_uint(b2), __float_as_uint(b3), 0x0040), 0x5410);
    }
}

// Offset, in the padded shared-memory row, of element base + j * S from element base, for the strides and
// alignments of the passes below (S = 32: base is the start of a 32 * R block, R <= 16; S = 512: any base).
template <int LOG_S>
__host__ __device__ constexpr int pad_step(int j) {
    return LOG_S == 9 ? 608 * j : 36 * j + ((j >> 3) << 4);
}

// CTAs are persistent: CTA b takes rows b, b + gridDim.x, ... (the SMs are filled once; a row's loads overlap the
// arithmetic of the other CTAs' rows -- staging the next row ahead of time, in registers or by cp.async into shared
// memory, was measured and lost: it costs registers or a CTA per SM).  The block has a whole number of warps; threads
// beyond K / 32 redo the last thread's work (same values to the same addresses), which keeps every branch uniform.
//   MID   1: a middle pass (strides 32 .. 256) precedes the last pass, whose first stride is then 512
//   R2    stages of the last pass (0: the first pass was the only one)
template <bool BF16_IN, bool UPPER_ONLY, int MID, int R2>
__global__ void __launch_bounds__(kRowsMaxThreads, 2)
quantize_rows_kernel(const void* __restrict__ X, int M, int K, int s0, float clip, float inv_sqrt_b, int8_t* __restrict__ q_a,
                     float* __restrict__ s_a) {
    constexpr int LOG_S = MID ? 9 : 5, S = 1 << LOG_S;
    constexpr int R = 1 << R2, C = 32 >> R2, P = C / 2;
    extern __shared__ __align__(16) float row[];
    __shared__ __align__(16) float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const int t = min(static_cast<int>(threadIdx.x), (K >> 5) - 1);
    const bool rotated = s0 > 0;
    // last pass: the thread's rows and columns
    int base = 32 * t;
    if (R2 > 0) {
        constexpr int LOG_CHUNKS = LOG_S + R2 - 5;  // S / C column chunks per block of S * R elements
        base = ((t >> LOG_CHUNKS) << (LOG_S + R2)) + (t & ((1 << LOG_CHUNKS) - 1)) * C;
    }
    const float* last_src = row + pad_index(base);
    float* mid_base = row + pad_index(((t >> 4) << 9) + 2 * (t & 15));
    ulonglong2* first_dst = reinterpret_cast<ulonglong2*>(row + pad_index(32 * t));

    constexpr int LOADS = BF16_IN ? 4 : 8;   // 16-byte pieces of the thread's 32 elements
    int parity = 0;
    for (int m = blockIdx.x; m < M; m += gridDim.x, parity ^= 1) {
        // ---- first pass: 32 contiguous elements, strides 1 .. 16
        f32x2_t pr[16];
        {
            float v[32];
            uint4 w4[LOADS];
            const uint4* src = reinterpret_cast<const uint4*>(static_cast<const unsigned char*>(X) + static_cast<size_t>(m) * K * (BF16_IN ? 2 : 4)) + LOADS * t;
#pragma unroll
            for (int i = 0; i < LOADS; ++i) w4[i] = __ldg(src + i);
            if constexpr (BF16_IN) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t w[4] = {w4[i].x, w4[i].y, w4[i].z, w4[i].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        v[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
                        v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                    }
                }
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    v[4 * i] = __uint_as_float(w4[i].x), v[4 * i + 1] = __uint_as_float(w4[i].y), v[4 * i + 2] = __uint_as_float(w4[i].z),
                    v[4 * i + 3] = __uint_as_float(w4[i].w);
            }
            if (s0 == 5) {  // the usual case, without per-stage tests
#pragma unroll
                for (int i = 0; i < 16; ++i) pr[i] = f2_make(__fadd_rn(v[2 * i], v[2 * i + 1]), __fsub_rn(v[2 * i], v[2 * i + 1]));
                butterfly_pairs<16>(pr, 4);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    pr[i] = (s0 > 0) ? f2_make(__fadd_rn(v[2 * i], v[2 * i + 1]), __fsub_rn(v[2 * i], v[2 * i + 1])) : f2_make(v[2 * i], v[2 * i + 1]);
                butterfly_pairs<16>(pr, s0 - 1);
            }
        }
        f32x2_t v[R][P];
        if constexpr (R2 == 0) {
#pragma unroll
            for (int i = 0; i < P; ++i) v[0][i] = pr[i];
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) first_dst[i] = make_ulonglong2(pr[2 * i], pr[2 * i + 1]);
            __syncthreads();
            if constexpr (MID) {
                // ---- middle pass: strides 32 .. 256, 16 rows x 2 neighbouring columns, in place
                f32x2_t w[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) w[j] = *reinterpret_cast<const f32x2_t*>(mid_base + pad_step<5>(j));
                butterfly_pairs<16>(w, 4);
#pragma unroll
                for (int j = 0; j < 16; ++j) *reinterpret_cast<f32x2_t*>(mid_base + pad_step<5>(j)) = w[j];
                __syncthreads();
            }
            // ---- last pass: R2 stages from stride S on R rows x C neighbouring columns, kept in registers.  (Its reads
            // precede the barrier of the row-scale reduction, so the next row's first pass cannot overwrite shared
            // memory that is still being read.)
#pragma unroll
            for (int j = 0; j < R; ++j) {
                const float* src = last_src + pad_step<LOG_S>(j);
                if constexpr (P == 1) {
                    v[j][0] = *reinterpret_cast<const f32x2_t*>(src);
                } else {
#pragma unroll
                    for (int i = 0; i < P / 2; ++i) {
                        const ulonglong2 f = reinterpret_cast<const ulonglong2*>(src)[i];
                        v[j][2 * i] = f.x, v[j][2 * i + 1] = f.y;
                    }
                }
            }
#pragma unroll
            for (int h = 1; h < R; h <<= 1)
#pragma unroll
                for (int j = 0; j < R; ++j)
                    if ((j & h) == 0) {
#pragma unroll
                        for (int i = 0; i < P; ++i) {
                            const f32x2_t a = v[j][i], b = v[j + h][i];
                            v[j][i] = f2_add(a, b);
                            v[j + h][i] = f2_sub(a, b);
                        }
                    }
        }
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < R; ++j)
#pragma unroll
            for (int i = 0; i < P; ++i) amax = max_abs2(v[j][i], amax);
        const RowScale sc = block_row_scale_wide(amax, clip, red, parity);
        if (threadIdx.x == 0) s_a[m] = rotated ? __fmul_rn(sc.s_u, inv_sqrt_b) : sc.s_u;
        // ---- quantize from the registers and store; one test per thread and row for "some element was near a
        // rounding tie", after which the thread redoes its elements with exact quotients (rare) and stores again
        int8_t* q_row = q_a + static_cast<size_t>(m) * K + base;
        auto store_row = [&](int j, const f32x2_t (&y)[P]) {
            uint32_t out[(P + 1) / 2];
            low_bytes<P>(y, out);
            int8_t* dst = q_row + j * S;
            if constexpr (C == 2) *reinterpret_cast<uint16_t*>(dst) = static_cast<uint16_t>(out[0]);
            else if constexpr (C == 4) *reinterpret_cast<uint32_t*>(dst) = out[0];
            else if constexpr (C == 8) *reinterpret_cast<uint2*>(dst) = make_uint2(out[0], out[1]);
            else {
#pragma unroll
                for (int i = 0; i < C / 16; ++i) reinterpret_cast<uint4*>(dst)[i] = make_uint4(out[4 * i], out[4 * i + 1], out[4 * i + 2], out[4 * i + 3]);
            }
        };
        float dmax = (sc.inv != 0.0f) ? 0.0f : 1.0f;
        const f32x2_t inv2 = f2_make(sc.inv, sc.inv);
#pragma unroll
        for (int j = 0; j < R; ++j) {
            f32x2_t y[P];
            quantize_pairs_fast<P, UPPER_ONLY>(v[j], inv2, y, dmax);
            store_row(j, y);
        }
        if (dmax > kTieGuard) {
#pragma unroll
            for (int j = 0; j < R; ++j) {
                f32x2_t y[P];
                quantize_pairs_exact<P>(v[j], sc.s_u, y);
                store_row(j, y);
            }
        }
    }
}

inline bool quantize_rows_supports(int K, int had_block) {
    if (K % 32 != 0 || K > 16384) return false;
    if (had_block <= 1) return true;
    return (had_block & (had_block - 1)) == 0 && had_block <= 8192 && K % had_block == 0;
}

}  // namespace qift

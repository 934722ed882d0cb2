// Blockwise Walsh-Hadamard rotation, fused per-token INT4 activation quantizer, offline rotation.
//
// One CTA per row.  The row lives in shared memory as fp32; the butterfly runs in radix-16 passes
// (four stages per pass in registers), stages in ascending stride so that every add/sub sees the
// same operands as the textbook in-place butterfly -- the result is then bit-identical to it
// whatever the thread mapping, because each stage is a set of independent IEEE additions.
#pragma once

#include "common.cuh"

namespace qift {

constexpr int kRowThreads = 256;
constexpr int kMaxRowK = 16384;

template <int R>
__device__ __forceinline__ void butterfly_regs(float (&v)[R], int active_stages) {
#pragma unroll
    for (int s = 0, h = 1; h < R; h <<= 1, ++s) {
        if (s < active_stages) {
#pragma unroll
            for (int i = 0; i < R; ++i) {
                if ((i & h) == 0) {
                    const float a = v[i], b = v[i + h];
                    v[i] = __fadd_rn(a, b);
                    v[i + h] = __fsub_rn(a, b);
                }
            }
        }
    }
}

// One radix-16 pass over the row in shared memory: strides sb, 2sb, 4sb, 8sb (those below B).
__device__ __forceinline__ void wht_pass_smem(float* row, int K, int sb, int B) {
    int stages = 0;
    for (int h = sb; h < B && stages < 4; h <<= 1) ++stages;
    const int R = 1 << stages;  // elements of one group
    const int groups = K / R;
    if (stages == 4) {
        for (int q = threadIdx.x; q < groups; q += blockDim.x) {
            const int base = (q / sb) * (16 * sb) + (q % sb);
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = row[base + j * sb];
            butterfly_regs<16>(v, 4);
#pragma unroll
            for (int j = 0; j < 16; ++j) row[base + j * sb] = v[j];
        }
    } else {  // last, partial pass: 2, 4 or 8 elements per group
        for (int q = threadIdx.x; q < groups; q += blockDim.x) {
            const int base = (q / sb) * (R * sb) + (q % sb);
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (j < R) ? row[base + j * sb] : 0.0f;
            butterfly_regs<8>(v, stages);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < R) row[base + j * sb] = v[j];
        }
    }
}

// Loads the row (fp32 or bf16), runs the strides 1..8 in registers, leaves the row in shared memory,
// then finishes the transform there.  B <= 1 means no rotation.
template <bool BF16_IN>
__device__ __forceinline__ void load_and_transform(const void* X, size_t row_index, int K, int B, float* row) {
    const int groups = K / 16;
    int stages0 = 0;
    for (int h = 1; h < B && stages0 < 4; h <<= 1) ++stages0;
    for (int q = threadIdx.x; q < groups; q += blockDim.x) {
        float v[16];
        if constexpr (BF16_IN) {
            const uint4* src = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(X) + row_index * K) + 2 * q;
            const uint4 a = src[0], b = src[1];
            const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[2 * i] = __uint_as_float(w[i] << 16);
                v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
            }
        } else {
            const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(X) + row_index * K) + 4 * q;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 f = src[i];
                v[4 * i] = f.x, v[4 * i + 1] = f.y, v[4 * i + 2] = f.z, v[4 * i + 3] = f.w;
            }
        }
        butterfly_regs<16>(v, stages0);
        float4* dst = reinterpret_cast<float4*>(row) + 4 * q;
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    }
    __syncthreads();
    for (int sb = 16; sb < B; sb *= 16) {
        wht_pass_smem(row, K, sb, B);
        __syncthreads();
    }
}

__device__ __forceinline__ float block_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, red[w]);
    __syncthreads();
    return r;
}

// K2: rotate + quantize one token row per CTA.
template <bool BF16_IN>
__global__ void __launch_bounds__(kRowThreads)
quantize_act_kernel(const void* __restrict__ X, int K, int B, float clip, float inv_sqrt_b,
                    int8_t* __restrict__ q_a, float* __restrict__ s_a) {
    extern __shared__ __align__(16) float row[];
    __shared__ float red[kRowThreads / 32];
    pdl_launch_dependents();
    pdl_wait();
    const size_t m = blockIdx.x;
    load_and_transform<BF16_IN>(X, m, K, B, row);

    const int groups = K / 16;
    float amax = 0.0f;
    for (int q = threadIdx.x; q < groups; q += blockDim.x) {
        const float4* src = reinterpret_cast<const float4*>(row) + 4 * q;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = src[i];
            amax = fmaxf(amax, fmaxf(fmaxf(fabsf(f.x), fabsf(f.y)), fmaxf(fabsf(f.z), fabsf(f.w))));
        }
    }
    amax = block_max(amax, red);
    float s_u = 1.0f;
    if (amax != 0.0f) s_u = __fdiv_rn(__fmul_rn(amax, clip), 7.0f);
    if (threadIdx.x == 0) s_a[m] = (B > 1) ? __fmul_rn(s_u, inv_sqrt_b) : s_u;

    for (int q = threadIdx.x; q < groups; q += blockDim.x) {
        const float4* src = reinterpret_cast<const float4*>(row) + 4 * q;
        uint32_t out[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = src[i];
            const float e[4] = {f.x, f.y, f.z, f.w};
            uint32_t w = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int v = __float2int_rn(__fdiv_rn(e[j], s_u));
                v = max(-8, min(7, v));
                w |= (static_cast<uint32_t>(v) & 0xffu) << (8 * j);
            }
            out[i] = w;
        }
        reinterpret_cast<uint4*>(q_a + m * K)[q] = make_uint4(out[0], out[1], out[2], out[3]);
    }
}

// S0: orthonormal blockwise rotation of fp32 rows.
__global__ void __launch_bounds__(kRowThreads)
rotate_rows_kernel(const float* __restrict__ X, int K, int B, float inv_sqrt_b, float* __restrict__ Y) {
    extern __shared__ __align__(16) float row[];
    pdl_launch_dependents();
    pdl_wait();
    const size_t m = blockIdx.x;
    load_and_transform<false>(X, m, K, B, row);
    for (int i = threadIdx.x; i < K / 4; i += blockDim.x) {
        float4 f = reinterpret_cast<const float4*>(row)[i];
        f.x = __fmul_rn(f.x, inv_sqrt_b), f.y = __fmul_rn(f.y, inv_sqrt_b);
        f.z = __fmul_rn(f.z, inv_sqrt_b), f.w = __fmul_rn(f.w, inv_sqrt_b);
        reinterpret_cast<float4*>(Y + m * K)[i] = f;
    }
}

}  // namespace qift

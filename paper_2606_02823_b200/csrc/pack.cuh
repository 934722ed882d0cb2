// Weight quantizer + packer (one CTA per output channel) and the unpacker used by tests.
#pragma once

#include "common.cuh"

namespace qift {

constexpr int kPackThreads = 256;
constexpr int kNumCandidates = 80;  // clipping ratios 1.00, 0.99, ..., 0.21

template <int LV>
__device__ __forceinline__ int nearest_code(float w, float s) {
    const float t = __fdiv_rn(w, s);
    if constexpr (LV == QIFT_LEVELS_MNZ) return (t > -2.0f) + (t > 0.0f) + (t > 2.0f);
    if constexpr (LV == QIFT_LEVELS_POT) return (t > -2.5f) + (t > 0.0f) + (t > 2.5f);
    if constexpr (LV == QIFT_LEVELS_SYM) return max(-2, min(1, __float2int_rn(t))) + 2;
    return max(-8, min(7, __float2int_rn(t))) & 15;
}

template <int LV>
__global__ void __launch_bounds__(kPackThreads)
pack_weights_kernel(const float* __restrict__ W, int N, int K, int mode, float* __restrict__ s_n,
                    uint32_t* __restrict__ packed) {
    extern __shared__ __align__(16) float row[];
    __shared__ float red[kPackThreads / 32];
    __shared__ double err[kNumCandidates][kPackThreads / 32];
    __shared__ float s_shared;
    // No early launch of dependents here: the product kernels prefetch packed weights before their
    // own dependency wait, which is only safe if whoever writes those weights has fully completed.
    pdl_wait();
    const size_t n = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pitch = packed_pitch(K, LV);
    if (n >= static_cast<size_t>(N)) {  // padding row of the last row block: zero words
        for (int u = tid; u < pitch / 4; u += blockDim.x)
            *reinterpret_cast<uint4*>(packed + packed_word_address(static_cast<int>(n), 4 * u, pitch)) = make_uint4(0, 0, 0, 0);
        return;
    }

    float amax = 0.0f;
    for (int i = tid; i < K / 4; i += blockDim.x) {
        const float4 f = reinterpret_cast<const float4*>(W + n * K)[i];
        reinterpret_cast<float4*>(row)[i] = f;
        amax = fmaxf(amax, fmaxf(fmaxf(fabsf(f.x), fabsf(f.y)), fmaxf(fabsf(f.z), fabsf(f.w))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) red[warp] = amax;
    __syncthreads();
    amax = red[0];
    for (int w = 1; w < kPackThreads / 32; ++w) amax = fmaxf(amax, red[w]);

    constexpr float g = top_level(LV);
    float s = 1.0f;
    if (mode == QIFT_SCALE_GIVEN) {
        s = s_n[n];
    } else if (amax != 0.0f) {
        if (mode == QIFT_SCALE_ABSMAX) {
            s = __fdiv_rn(amax, g);
        } else {
            // Squared error of every candidate scale; per-element terms are formed exactly as
            // d = w - s*level, d*d in fp64 without contraction, partial sums per thread in
            // ascending k, then a fixed-order tree.
            for (int c0 = 0; c0 < kNumCandidates; c0 += 8) {
                float sc[8];
                double e[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float p = __fdiv_rn(static_cast<float>(100 - (c0 + j)), 100.0f);
                    sc[j] = __fdiv_rn(__fmul_rn(p, amax), g);
                    e[j] = 0.0;
                }
                for (int k = tid; k < K; k += blockDim.x) {
                    const float w = row[k];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int code = nearest_code<LV>(w, sc[j]);
                        const double rec = __dmul_rn(static_cast<double>(sc[j]), static_cast<double>(level_from_code<LV>(code)));
                        const double d = __dsub_rn(static_cast<double>(w), rec);
                        e[j] = __dadd_rn(e[j], __dmul_rn(d, d));
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    double v = e[j];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
                    if (lane == 0) err[c0 + j][warp] = v;
                }
            }
            __syncthreads();
            if (tid == 0) {
                int best = 0;
                double best_e = 0.0;
                for (int i = 0; i < kNumCandidates; ++i) {
                    double v = 0.0;
                    for (int w = 0; w < kPackThreads / 32; ++w) v = __dadd_rn(v, err[i][w]);
                    if (i == 0 || v < best_e) best_e = v, best = i;
                }
                const float p = __fdiv_rn(static_cast<float>(100 - best), 100.0f);
                s_shared = __fdiv_rn(__fmul_rn(p, amax), g);
            }
            __syncthreads();
            s = s_shared;
        }
    }
    if (tid == 0 && mode != QIFT_SCALE_GIVEN) s_n[n] = s;

    constexpr int PER = codes_per_word(LV);
    constexpr int BITS = 32 / PER;
    const int words = K / PER;
    for (int u = tid; u < pitch / 4; u += blockDim.x) {  // one 16-byte group of four words per thread
        uint32_t out[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = 4 * u + e;
            uint32_t w = 0;
            if (j < words) {
#pragma unroll
                for (int r = 0; r < PER; ++r) {
                    const int t = r / 4, b = r % 4;
                    w |= static_cast<uint32_t>(nearest_code<LV>(row[j * PER + r], s)) << (8 * b + BITS * t);
                }
            }
            out[e] = w;
        }
        *reinterpret_cast<uint4*>(packed + packed_word_address(static_cast<int>(n), 4 * u, pitch)) =
            make_uint4(out[0], out[1], out[2], out[3]);
    }
}

__global__ void unpack_codes_kernel(const uint32_t* __restrict__ packed, long long total, int K, int per,
                                    uint8_t* __restrict__ codes) {
    pdl_launch_dependents();
    pdl_wait();
    const int bits = 32 / per;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long n = i / K;
        const int k = static_cast<int>(i % K);
        const int j = k / per, r = k % per, t = r / 4, b = r % 4;
        const uint32_t w = packed[packed_word_address(static_cast<int>(n), j, round_up16(K / per))];
        codes[i] = static_cast<uint8_t>((w >> (8 * b + bits * t)) & ((1u << bits) - 1u));
    }
}

}  // namespace qift

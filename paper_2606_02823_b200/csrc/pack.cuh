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
    if constexpr (LV == QIFT_LEVELS_INT3) return max(-4, min(3, __float2int_rn(t))) & 7;
    return max(-8, min(7, __float2int_rn(t))) & 15;
}

// Division-free nearest level for one scale, bit-identical to nearest_code().
//   No-zero sets: the decision t > theta with t = fl(w / s) equals |w| > fl(theta * s) unless |w| lies
//   within 2^-20 (relative) of that product -- roundings of the product and of the quotient move either
//   side by at most 2^-23 -- and t > 0 equals w > 0 unless the quotient underflows; in those (rare)
//   cases the division decides.
//   Integer sets: t = w * (1/s) differs from the quotient by < 2^-19 for |t| <= 8, so both round to the
//   same integer unless t lies within 2^-17 of a tie; clamp before rounding = clamp after.
template <int LV>
struct LevelCoder {
    float s, thr, band, tiny, inv;
    __device__ __forceinline__ void init(float scale) {
        s = scale;
        constexpr float theta = (LV == QIFT_LEVELS_POT) ? 2.5f : 2.0f;
        thr = __fmul_rn(theta, scale);
        band = __fmul_rn(thr, 9.5367431640625e-07f);  // 2^-20
        tiny = __fmul_rn(scale, 7.888609052210118e-31f);  // 2^-100
        inv = (scale >= 1e-30f && scale <= 1e30f) ? __fdiv_rn(1.0f, scale) : 0.0f;
    }
    // Branch-free part: code of w and, in `mag`, |level| for the no-zero sets / the signed level for the
    // integer sets; `unsure` is set when the division has to decide (then use exact()).
    __device__ __forceinline__ int fast(float w, float& mag, bool& unsure) const {
        if constexpr (LV == QIFT_LEVELS_MNZ || LV == QIFT_LEVELS_POT) {
            const float a = fabsf(w);
            unsure = unsure || fabsf(__fsub_rn(a, thr)) <= band || (a != 0.0f && a < tiny);
            const bool outer = a > thr;
            mag = outer ? top_level(LV) : 1.0f;
            return (w > 0.0f) ? 2 + static_cast<int>(outer) : 1 - static_cast<int>(outer);
        } else {
            constexpr float lo = (LV == QIFT_LEVELS_SYM) ? -2.0f : (LV == QIFT_LEVELS_INT3) ? -4.0f : -8.0f;
            constexpr float hi = (LV == QIFT_LEVELS_SYM) ? 1.0f : (LV == QIFT_LEVELS_INT3) ? 3.0f : 7.0f;
            const float t = fminf(fmaxf(__fmul_rn(w, inv), lo), hi);
            const float r = __fsub_rn(__fadd_rn(t, 12582912.0f), 12582912.0f);
            unsure = unsure || inv == 0.0f || fabsf(__fsub_rn(t, r)) > 0.49999237f;
            mag = r;
            const int q = static_cast<int>(r);
            return (LV == QIFT_LEVELS_SYM) ? q + 2 : (LV == QIFT_LEVELS_INT3) ? (q & 7) : (q & 15);
        }
    }
    __device__ __forceinline__ int exact(float w, float& mag) const {
        const int c = nearest_code<LV>(w, s);
        const float lv = static_cast<float>(level_from_code<LV>(c));
        mag = (LV == QIFT_LEVELS_MNZ || LV == QIFT_LEVELS_POT) ? fabsf(lv) : lv;
        return c;
    }
};

template <int LV>
__global__ void __launch_bounds__(kPackThreads)
pack_weights_kernel(const float* __restrict__ W, int N, int K, int mode, float* __restrict__ s_n,
                    uint32_t* __restrict__ packed) {
    extern __shared__ __align__(16) float row[];
    __shared__ float red[kPackThreads / 32];
    __shared__ double err[kNumCandidates][kPackThreads / 32];
    __shared__ double mom[2][kPackThreads / 32];
    __shared__ float cand[kNumCandidates];
    __shared__ unsigned long long bin_sum[kNumCandidates];
    __shared__ int bin_cnt[kNumCandidates];
    __shared__ float s_shared;
    // No early launch of dependents here: the product kernels prefetch packed weights before their
    // own dependency wait, which is only safe if whoever writes those weights has fully completed.
    pdl_wait();
    const size_t n = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pitch = packed_pitch(K, LV);
    if (n >= static_cast<size_t>(N)) {  // padding row of the last row block: zero words
        for (int u = tid; u < pitch / 4; u += blockDim.x) {
            if constexpr (LV == QIFT_LEVELS_INT3) {
                *reinterpret_cast<uint4*>(packed + int3_low_address(static_cast<int>(n), 4 * u, pitch)) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint2*>(packed + int3_high_address(static_cast<int>(n), 4 * u, pitch)) = make_uint2(0, 0);
            } else {
                *reinterpret_cast<uint4*>(packed + packed_word_address(static_cast<int>(n), 4 * u, pitch)) = make_uint4(0, 0, 0, 0);
            }
        }
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
            constexpr bool kNoZero = (LV == QIFT_LEVELS_MNZ || LV == QIFT_LEVELS_POT);
            if constexpr (kNoZero) {
                // No-zero sets {+-1, +-top}: a weight's level has its sign and magnitude 1 (inner) or top
                // (outer, |w| / s > theta), so with a = |w| the squared error of a candidate scale s is
                //   E(s) = sum a^2 - 2 s (sum a + (top-1) sum_outer a) + s^2 (K + (top^2-1) n_outer),
                // and because the candidate scales decrease, a weight that is outer for candidate j is outer
                // for every later one.  So each weight is looked at ONCE: its switch index b (the first
                // candidate for which it is outer) is found from the table of thresholds (a first guess
                // from the ratio, corrected by comparisons; decided by the division where |w| is within
                // 2^-20 of a threshold), and its magnitude and a count go into bin b.  Outer sums and
                // counts of all 80 candidates are prefix sums over the bins.  The magnitudes are added as
                // 64-bit fixed-point integers scaled by the row's maximum (outer weights are >= 0.14 max, so
                // they are represented exactly and the shared-memory atomics give the same sum in any
                // order); sum a and sum a^2 are fp64, per thread in ascending k, then fixed-order trees.
                // The regrouping changes E by ~1e-15 relative, far inside the 1e-12 within which two
                // candidates count as tied.
                constexpr double top = top_level(LV);
                float* thr = cand;  // [kNumCandidates] thresholds theta * s_j, decreasing in j
                for (int j = tid; j < kNumCandidates; j += blockDim.x) {
                    LevelCoder<LV> c;
                    c.init(__fdiv_rn(__fmul_rn(__fdiv_rn(static_cast<float>(100 - j), 100.0f), amax), g));
                    thr[j] = c.thr;
                    bin_sum[j] = 0ull, bin_cnt[j] = 0;
                }
                __syncthreads();
                int ex;
                frexpf(amax, &ex);                              // amax < 2^ex
                const double to_fixed = ldexp(1.0, 48 - ex);    // a * to_fixed < 2^48, exact for a >= amax * 2^-24
                const float ratio = __fdiv_rn(g, __fmul_rn((LV == QIFT_LEVELS_POT) ? 2.5f : 2.0f, amax));
                double a2 = 0.0, a1 = 0.0;
                for (int k = tid; k < K; k += blockDim.x) {
                    const float w = row[k];
                    const float a = fabsf(w);
                    const double ad = static_cast<double>(a);
                    a2 = __dadd_rn(a2, __dmul_rn(ad, ad));
                    a1 = __dadd_rn(a1, ad);
                    // first guess: a > theta p_j amax / g  <=>  (100 - j) / 100 < a g / (theta amax)
                    int bsw = min(kNumCandidates, max(0, 101 - static_cast<int>(100.0f * a * ratio)));
                    while (bsw > 0 && a > thr[bsw - 1]) --bsw;
                    while (bsw < kNumCandidates && !(a > thr[bsw])) ++bsw;
                    // |w| within 2^-20 of a neighbouring threshold: the division decides (monotone in j)
                    if (bsw > 0 && __fsub_rn(thr[bsw - 1], a) <= thr[bsw - 1] * 9.5367431640625e-07f) {
                        while (bsw > 0) {
                            float mag;
                            LevelCoder<LV> c;
                            c.init(__fdiv_rn(__fmul_rn(__fdiv_rn(static_cast<float>(100 - (bsw - 1)), 100.0f), amax), g));
                            c.exact(w, mag);
                            if (mag == 1.0f) break;
                            --bsw;
                        }
                    }
                    if (bsw < kNumCandidates && __fsub_rn(a, thr[bsw]) <= thr[bsw] * 9.5367431640625e-07f) {
                        while (bsw < kNumCandidates) {
                            float mag;
                            LevelCoder<LV> c;
                            c.init(__fdiv_rn(__fmul_rn(__fdiv_rn(static_cast<float>(100 - bsw), 100.0f), amax), g));
                            c.exact(w, mag);
                            if (mag != 1.0f) break;
                            ++bsw;
                        }
                    }
                    if (bsw < kNumCandidates) {
                        atomicAdd(&bin_sum[bsw], static_cast<unsigned long long>(__dmul_rn(ad, to_fixed)));
                        atomicAdd(&bin_cnt[bsw], 1);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    a2 = __dadd_rn(a2, __shfl_xor_sync(0xffffffffu, a2, o));
                    a1 = __dadd_rn(a1, __shfl_xor_sync(0xffffffffu, a1, o));
                }
                if (lane == 0) mom[0][warp] = a2, mom[1][warp] = a1;
                __syncthreads();
                if (tid < kNumCandidates) {  // E of candidate tid, left in err[tid][0]
                    double A = 0.0, S = 0.0;
                    for (int w = 0; w < kPackThreads / 32; ++w) A = __dadd_rn(A, mom[0][w]), S = __dadd_rn(S, mom[1][w]);
                    unsigned long long so = 0;
                    int n_out = 0;
                    for (int b = 0; b <= tid; ++b) so += bin_sum[b], n_out += bin_cnt[b];
                    const double So = ldexp(static_cast<double>(so), ex - 48);
                    const float p = __fdiv_rn(static_cast<float>(100 - tid), 100.0f);
                    const double sj = static_cast<double>(__fdiv_rn(__fmul_rn(p, amax), g));
                    const double lin = S + (top - 1.0) * So;
                    const double quad = static_cast<double>(K) + (top * top - 1.0) * static_cast<double>(n_out);
                    err[tid][0] = A - 2.0 * sj * lin + sj * sj * quad;  // each thread touches its own row of err only
#pragma unroll
                    for (int w = 1; w < kPackThreads / 32; ++w) err[tid][w] = 0.0;
                }
            } else {
                // Integer sets (Eq. 1): level q = clamp(rint(w / s)).  |q| is the number of boundaries
                // m + 1/2 (m = 0, 1, ...) that |w| / s has crossed, up to 7 (1) on the positive and 8 (2)
                // on the negative side for INT4 (the standard W2 set), and w q = |w| |q|, q^2 = sum over
                // the crossed boundaries of 2m + 1.  So
                //   E(s) = sum w^2 - 2 s sum_{crossings} |w| + s^2 sum_{crossings} (2m + 1),
                // and as for the no-zero sets a crossing, once made, stays for every later (smaller)
                // candidate scale: each (weight, boundary) pair is binned once at its switch index and the
                // two sums of every candidate are prefix sums over the bins.  Decisions within 2^-20 of a
                // boundary (where round-half-even and the rounding of the quotient matter) are taken with
                // the division.  |w| enters as an exact 64-bit fixed-point integer (crossing weights are
                // >= 0.015 max); pairs that have switched at the first candidate already -- the majority --
                // are summed per thread first.
                constexpr int kLimPos = (LV == QIFT_LEVELS_SYM) ? 1 : (LV == QIFT_LEVELS_INT3) ? 3 : 7;
                constexpr int kLimNeg = (LV == QIFT_LEVELS_SYM) ? 2 : (LV == QIFT_LEVELS_INT3) ? 4 : 8;
                float* sj = cand;  // [kNumCandidates] candidate scales, decreasing in j
                for (int j = tid; j < kNumCandidates; j += blockDim.x) {
                    sj[j] = __fdiv_rn(__fmul_rn(__fdiv_rn(static_cast<float>(100 - j), 100.0f), amax), g);
                    bin_sum[j] = 0ull, bin_cnt[j] = 0;
                }
                __syncthreads();
                int ex;
                frexpf(amax, &ex);                              // amax < 2^ex
                const double to_fixed = ldexp(1.0, 44 - ex);    // |w| * to_fixed < 2^44
                const float guess = __fdiv_rn(100.0f * g, amax);
                const float s_last = sj[kNumCandidates - 1];
                double a2 = 0.0;
                unsigned long long first_sum = 0;
                int first_cnt = 0;
                auto crossed = [&](float w, int j, int m) {  // exact: has |q| reached m + 1 at candidate j
                    const int lv = level_from_code<LV>(nearest_code<LV>(w, sj[j]));
                    return abs(lv) >= m + 1;
                };
                for (int k = tid; k < K; k += blockDim.x) {
                    const float w = row[k];
                    const float a = fabsf(w);
                    const double ad = static_cast<double>(a);
                    a2 = __dadd_rn(a2, __dmul_rn(ad, ad));
                    const unsigned long long fx = static_cast<unsigned long long>(__dmul_rn(ad, to_fixed));
                    const int lim = (w < 0.0f) ? kLimNeg : kLimPos;
                    for (int m = 0; m < lim; ++m) {
                        const float h = static_cast<float>(m) + 0.5f;
                        if (a < __fmul_rn(__fmul_rn(h, s_last), 0.999999f)) break;  // never crossed, nor the later ones
                        // first guess: a > h p_j amax / g  <=>  (100 - j) < 100 a g / (h amax)
                        int bsw = min(kNumCandidates, max(0, 101 - static_cast<int>(__fdiv_rn(a * guess, h))));
                        while (bsw > 0 && a > __fmul_rn(h, sj[bsw - 1])) --bsw;
                        while (bsw < kNumCandidates && !(a > __fmul_rn(h, sj[bsw]))) ++bsw;
                        if (bsw > 0) {
                            const float t = __fmul_rn(h, sj[bsw - 1]);
                            if (__fsub_rn(t, a) <= t * 9.5367431640625e-07f)
                                while (bsw > 0 && crossed(w, bsw - 1, m)) --bsw;
                        }
                        if (bsw < kNumCandidates) {
                            const float t = __fmul_rn(h, sj[bsw]);
                            if (__fsub_rn(a, t) <= t * 9.5367431640625e-07f)
                                while (bsw < kNumCandidates && !crossed(w, bsw, m)) ++bsw;
                        }
                        if (bsw == 0) {
                            first_sum += fx, first_cnt += 2 * m + 1;
                        } else if (bsw < kNumCandidates) {
                            atomicAdd(&bin_sum[bsw], fx);
                            atomicAdd(&bin_cnt[bsw], 2 * m + 1);
                        }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    a2 = __dadd_rn(a2, __shfl_xor_sync(0xffffffffu, a2, o));
                    first_sum += __shfl_xor_sync(0xffffffffu, first_sum, o);
                    first_cnt += __shfl_xor_sync(0xffffffffu, first_cnt, o);
                }
                if (lane == 0) {
                    mom[0][warp] = a2;
                    atomicAdd(&bin_sum[0], first_sum);
                    atomicAdd(&bin_cnt[0], first_cnt);
                }
                __syncthreads();
                if (tid < kNumCandidates) {  // E of candidate tid, left in err[tid][0]
                    double A = 0.0;
                    for (int w = 0; w < kPackThreads / 32; ++w) A = __dadd_rn(A, mom[0][w]);
                    unsigned long long ps = 0;
                    long long pq = 0;
                    for (int bb = 0; bb <= tid; ++bb) ps += bin_sum[bb], pq += bin_cnt[bb];
                    const double P = ldexp(static_cast<double>(ps), ex - 44);
                    const double sd = static_cast<double>(sj[tid]);
                    err[tid][0] = A - 2.0 * sd * P + sd * sd * static_cast<double>(pq);  // each thread touches its own row of err only
#pragma unroll
                    for (int w = 1; w < kPackThreads / 32; ++w) err[tid][w] = 0.0;
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

    // Codes: first one byte per weight into shared memory (threads stride over k: conflict-free), then
    // one packed word per thread from 16 consecutive code bytes -- with the bit layout of the packed
    // word four code bytes (k = 4t .. 4t+3) shifted left by 2t (4t for INT4) ARE plane t of the word --
    // and the four words of a 16-byte group are gathered in its first lane for one 128-bit store.
    constexpr int PER = codes_per_word(LV);
    const int words = K / PER;
    unsigned char* code_bytes = reinterpret_cast<unsigned char*>(row + K);
    LevelCoder<LV> final_coder;
    final_coder.init(s);
    __syncthreads();
    for (int k = tid; k < K; k += blockDim.x) {
        float mag;
        bool unsure = false;
        int c = final_coder.fast(row[k], mag, unsure);
        if (unsure) c = final_coder.exact(row[k], mag);
        code_bytes[k] = static_cast<unsigned char>(c);
    }
    __syncthreads();
    for (int j0 = 0; j0 < pitch; j0 += blockDim.x) {  // pitch is a multiple of 16, blockDim of 32: whole groups per warp
        const int j = j0 + tid;
        uint32_t w = 0, h = 0;
        if (j < words) {
            if constexpr (LV == QIFT_LEVELS_INT3) {
                // low plane: the two low bits as a two-bit word; high plane: this word's half of the shared high word
                const uint4 c = *reinterpret_cast<const uint4*>(code_bytes + 16 * j);
                constexpr uint32_t m2 = 0x03030303u, m1 = 0x01010101u;
                w = (c.x & m2) | ((c.y & m2) << 2) | ((c.z & m2) << 4) | ((c.w & m2) << 6);
                h = (((c.x >> 2) & m1) << int3_high_shift(j, 0)) | (((c.y >> 2) & m1) << int3_high_shift(j, 1)) |
                    (((c.z >> 2) & m1) << int3_high_shift(j, 2)) | (((c.w >> 2) & m1) << int3_high_shift(j, 3));
            } else if constexpr (PER == 16) {
                const uint4 c = *reinterpret_cast<const uint4*>(code_bytes + 16 * j);
                w = c.x | (c.y << 2) | (c.z << 4) | (c.w << 6);
            } else {
                const uint2 c = *reinterpret_cast<const uint2*>(code_bytes + 8 * j);
                w = c.x | (c.y << 4);
            }
        }
        const uint32_t w1 = __shfl_down_sync(0xffffffffu, w, 1), w2 = __shfl_down_sync(0xffffffffu, w, 2),
                       w3 = __shfl_down_sync(0xffffffffu, w, 3);
        if constexpr (LV == QIFT_LEVELS_INT3) {
            const uint32_t h1 = __shfl_down_sync(0xffffffffu, h, 1), h2 = __shfl_down_sync(0xffffffffu, h, 2),
                           h3 = __shfl_down_sync(0xffffffffu, h, 3);
            if ((tid & 3) == 0 && j < pitch) {
                *reinterpret_cast<uint4*>(packed + int3_low_address(static_cast<int>(n), j, pitch)) = make_uint4(w, w1, w2, w3);
                *reinterpret_cast<uint2*>(packed + int3_high_address(static_cast<int>(n), j, pitch)) = make_uint2(h | h1, h2 | h3);
            }
        } else {
            if ((tid & 3) == 0 && j < pitch)
                *reinterpret_cast<uint4*>(packed + packed_word_address(static_cast<int>(n), j, pitch)) = make_uint4(w, w1, w2, w3);
        }
    }
}

__global__ void unpack_codes_kernel(const uint32_t* __restrict__ packed, long long total, int K, int per, int three_bit,
                                    uint8_t* __restrict__ codes) {
    pdl_launch_dependents();
    pdl_wait();
    const int bits = 32 / per;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long n = i / K;
        const int k = static_cast<int>(i % K);
        const int j = k / per, r = k % per, t = r / 4, b = r % 4;
        if (three_bit) {
            const int pitch = round_up16(K / 16);
            const uint32_t lo = packed[int3_low_address(static_cast<int>(n), j, pitch)];
            const uint32_t hi = packed[int3_high_address(static_cast<int>(n), j, pitch)];
            codes[i] = static_cast<uint8_t>(((lo >> (8 * b + 2 * t)) & 3u) | (((hi >> (8 * b + int3_high_shift(j, t))) & 1u) << 2));
            continue;
        }
        const uint32_t w = packed[packed_word_address(static_cast<int>(n), j, round_up16(K / per))];
        codes[i] = static_cast<uint8_t>((w >> (8 * b + bits * t)) & ((1u << bits) - 1u));
    }
}

}  // namespace qift

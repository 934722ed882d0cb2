// KV4: asymmetric 4-bit key / value cache (Sec. 4.1: "asymmetric key and value quantization with
// clipping ratios of 0.95") and the single-query decode attention that reads it.
//
// Cache layout (device memory, owned by the caller), head-major so that the tokens of one KV head are
// contiguous:  codes uint8 [Hkv][T_cap][D/2] (two codes per byte, even dimension in the low nibble),
// scale fp32 [Hkv][T_cap], zero fp32 [Hkv][T_cap] (the integer zero-point 0..15 as a float).
// D = 128 (the head dimension of the LLaMA models the paper evaluates).
#pragma once

#include "common.cuh"

namespace qift {

constexpr int kKvD = 128;            // head dimension
constexpr int kKvRowBytes = kKvD / 2;

// ------------------------------------------------------------------------------------------------
// quantizer: one warp per (token, head) vector, four elements per lane
// ------------------------------------------------------------------------------------------------
// The rotation (B = 128, optional) is the same natural-order butterfly as everywhere else: strides 1
// and 2 inside a lane, strides 4..64 against the lane whose index differs in that bit -- the lower
// element of a pair takes a + b, the upper a - b, exactly the operands of the in-place butterfly, so
// the result is bit-identical to it.  Then one multiply by 1/sqrt(B) (orthonormal: queries carry no
// per-vector scale the factor could be folded into).
template <bool BF16_IN>
__global__ void __launch_bounds__(256)
kv4_quantize_kernel(const void* __restrict__ X, long long rows, int H, int had_block, float inv_sqrt_b, float clip, int t0,
                    int T_cap, uint8_t* __restrict__ codes, float* __restrict__ scale, float* __restrict__ zero) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long r = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);  // input row = token * H + head
    if (r >= rows) return;
    float v[4];
    if constexpr (BF16_IN) {
        const uint2 w = reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(X) + r * kKvD)[lane];
        v[0] = __uint_as_float(w.x << 16), v[1] = __uint_as_float(w.x & 0xffff0000u);
        v[2] = __uint_as_float(w.y << 16), v[3] = __uint_as_float(w.y & 0xffff0000u);
    } else {
        const float4 f = reinterpret_cast<const float4*>(static_cast<const float*>(X) + r * kKvD)[lane];
        v[0] = f.x, v[1] = f.y, v[2] = f.z, v[3] = f.w;
    }
    if (had_block > 1) {
        // element index = 4 * lane + e; strides below had_block only
        if (had_block > 1) {
            const float a0 = v[0], a1 = v[1], a2 = v[2], a3 = v[3];
            v[0] = __fadd_rn(a0, a1), v[1] = __fsub_rn(a0, a1), v[2] = __fadd_rn(a2, a3), v[3] = __fsub_rn(a2, a3);
        }
        if (had_block > 2) {
            const float a0 = v[0], a1 = v[1], a2 = v[2], a3 = v[3];
            v[0] = __fadd_rn(a0, a2), v[2] = __fsub_rn(a0, a2), v[1] = __fadd_rn(a1, a3), v[3] = __fsub_rn(a1, a3);
        }
        for (int h = 4; h < had_block; h <<= 1) {
            const int bit = h >> 2;  // lane bit of this stride
            const bool upper = (lane & bit) != 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float other = __shfl_xor_sync(0xffffffffu, v[e], bit);
                v[e] = upper ? __fsub_rn(other, v[e]) : __fadd_rn(v[e], other);
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = __fmul_rn(v[e], inv_sqrt_b);
    }
    float mn = fminf(fminf(fminf(v[0], v[1]), fminf(v[2], v[3])), 0.0f);
    float mx = fmaxf(fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3])), 0.0f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const float lo = __fmul_rn(mn, clip), hi = __fmul_rn(mx, clip);
    float s = 1.0f, z = 0.0f;
    if (hi != lo) {
        s = __fdiv_rn(__fsub_rn(hi, lo), 15.0f);
        z = rintf(__fdiv_rn(-lo, s));
    }
    const int zi = static_cast<int>(z);
    uint32_t packed = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int c = max(0, min(15, __float2int_rn(__fdiv_rn(v[e], s)) + zi));
        packed |= static_cast<uint32_t>(c) << (4 * e);
    }
    const long long t = r / H;
    const int h = static_cast<int>(r - t * H);
    const size_t slot = static_cast<size_t>(h) * T_cap + t0 + t;
    reinterpret_cast<uint16_t*>(codes + slot * kKvRowBytes)[lane] = static_cast<uint16_t>(packed);
    if (lane == 0) {
        scale[slot] = s;
        zero[slot] = z;
    }
}

// ------------------------------------------------------------------------------------------------
// decode attention over the 4-bit cache
// ------------------------------------------------------------------------------------------------
// out[h] = sum_t softmax_t(q[h] . Khat[t] / sqrt(D)) Vhat[t],  Khat = ks (kc - kz),  Vhat = vs (vc - vz),
// for the G = Hq / Hkv query heads that share a KV head.  fp32 throughout.
//
// Grid (head groups, splits, Hkv): a CTA takes a contiguous range of tokens of one KV head for G of the
// query heads that share it (G <= 2: more accumulators per thread would leave one CTA per SM; the head
// groups of a split run side by side and the second finds the codes in L2); eight warps take runs of
// four-token tiles in turn.  A lane is (token j of the tile, 16-dimension chunk c): it loads the 8
// bytes of codes of its chunk (a warp reads 256 contiguous bytes), turns them into floats ONCE and
// uses them for all G heads.  The zero-points never touch the per-element path:
//   q . Khat = ks (sum_d c_d q_d - kz sum_d q_d),     sum_t w_t Vhat_t = sum_t w_t vs_t c_t - (sum_t w_t vs_t vz_t).
// Softmax is the usual running-max form; partial (max, denominator, numerator) triples are merged
// across lanes, warps and finally splits (kv4_attention_combine_kernel).
struct Kv4Params {
    const float* q;  // [Hq][D]
    const uint8_t* k_codes;
    const float* k_scale;
    const float* k_zero;
    const uint8_t* v_codes;
    const float* v_scale;
    const float* v_zero;
    float* partial;  // [Hq][splits][D + 2]: numerator, running max, denominator
    float* out;      // [Hq][D]
    int T, T_cap, Hq, Hkv, splits, tokens_per_split;
    int heads_per_kv;  // Hq / Hkv
    float inv_sqrt_d;
};

constexpr int kKvWarps = 8;
constexpr int kKvUnroll = 2;  // four-token tiles a warp loads ahead (more costs the second CTA per SM)
constexpr int kKvPartial = kKvD + 2;

// Eight codes of a 32-bit word as floats: 2^23 + c has the code in its low mantissa bits.
__device__ __forceinline__ void nibbles_to_floats(uint32_t w, float (&f)[8]) {
    const uint32_t lo = w & 0x0f0f0f0fu, hi = (w >> 4) & 0x0f0f0f0fu;
    constexpr uint32_t magic = 0x4b000000u;  // 2^23
    f[0] = __uint_as_float(__byte_perm(lo, magic, 0x7440)) - 8388608.0f;
    f[1] = __uint_as_float(__byte_perm(hi, magic, 0x7440)) - 8388608.0f;
    f[2] = __uint_as_float(__byte_perm(lo, magic, 0x7441)) - 8388608.0f;
    f[3] = __uint_as_float(__byte_perm(hi, magic, 0x7441)) - 8388608.0f;
    f[4] = __uint_as_float(__byte_perm(lo, magic, 0x7442)) - 8388608.0f;
    f[5] = __uint_as_float(__byte_perm(hi, magic, 0x7442)) - 8388608.0f;
    f[6] = __uint_as_float(__byte_perm(lo, magic, 0x7443)) - 8388608.0f;
    f[7] = __uint_as_float(__byte_perm(hi, magic, 0x7443)) - 8388608.0f;
}

template <int G>
__global__ void __launch_bounds__(32 * kKvWarps)
kv4_attention_partial_kernel(const Kv4Params p) {
    __shared__ __align__(16) float qs[G][kKvD];       // q / sqrt(D)
    __shared__ float qsum[G][8];                       // its chunk sums
    __shared__ float red[kKvWarps][G][kKvPartial];
    pdl_launch_dependents();
    pdl_wait();
    const int kv = blockIdx.z, split = blockIdx.y;
    const int head0 = kv * p.heads_per_kv + blockIdx.x * G;  // first query head of this CTA
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = lane >> 3, c = lane & 7;

    for (int i = threadIdx.x; i < G * kKvD; i += blockDim.x)
        qs[i / kKvD][i % kKvD] = __fmul_rn(p.q[static_cast<size_t>(head0) * kKvD + i], p.inv_sqrt_d);
    __syncthreads();
    if (threadIdx.x < G * 8) {
        const int g = threadIdx.x >> 3, cc = threadIdx.x & 7;
        float s = 0.0f;
        for (int i = 0; i < 16; ++i) s += qs[g][16 * cc + i];
        qsum[g][cc] = s;
    }
    __syncthreads();

    const int t_begin = split * p.tokens_per_split;
    const int t_end = min(p.T, t_begin + p.tokens_per_split);
    const size_t head_row = static_cast<size_t>(kv) * p.T_cap;

    float m[G], l[G], zacc[G], acc[G][16];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY, l[g] = 0.0f, zacc[g] = 0.0f;
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[g][i] = 0.0f;
    }

    // kKvUnroll tiles per trip, all their loads issued before the first is used (a warp otherwise waits
    // out the full memory latency once per tile)
    for (int tb = t_begin + 4 * kKvUnroll * warp; tb < t_end; tb += 4 * kKvUnroll * kKvWarps) {
        uint2 kw[kKvUnroll], vw[kKvUnroll];
        float ks[kKvUnroll], kz[kKvUnroll], vs[kKvUnroll], vz[kKvUnroll];
#pragma unroll
        for (int u = 0; u < kKvUnroll; ++u) {
            const int t = tb + 4 * u + j;
            const size_t row = head_row + (t < t_end ? t : t_begin);
            kw[u] = *reinterpret_cast<const uint2*>(p.k_codes + row * kKvRowBytes + 8 * c);
            vw[u] = *reinterpret_cast<const uint2*>(p.v_codes + row * kKvRowBytes + 8 * c);
            ks[u] = p.k_scale[row], kz[u] = p.k_zero[row], vs[u] = p.v_scale[row], vz[u] = p.v_zero[row];
        }
#pragma unroll
        for (int u = 0; u < kKvUnroll; ++u) {
            if (tb + 4 * u >= t_end) break;  // warp-uniform: no token of this tile exists
            const bool valid = tb + 4 * u + j < t_end;
            float kd[16], vd[16];
            {
                float a[8], b[8];
                nibbles_to_floats(kw[u].x, a), nibbles_to_floats(kw[u].y, b);
#pragma unroll
                for (int i = 0; i < 8; ++i) kd[i] = a[i], kd[8 + i] = b[i];
                nibbles_to_floats(vw[u].x, a), nibbles_to_floats(vw[u].y, b);
#pragma unroll
                for (int i = 0; i < 8; ++i) vd[i] = a[i], vd[8 + i] = b[i];
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float4* qv = reinterpret_cast<const float4*>(&qs[g][16 * c]);
                float p0 = 0.0f, p1 = 0.0f, p2 = 0.0f, p3 = 0.0f;  // four independent chains
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 f = qv[i];
                    p0 = fmaf(kd[4 * i], f.x, p0), p1 = fmaf(kd[4 * i + 1], f.y, p1);
                    p2 = fmaf(kd[4 * i + 2], f.z, p2), p3 = fmaf(kd[4 * i + 3], f.w, p3);
                }
                float part = (p0 + p1) + (p2 + p3);
                part = fmaf(-kz[u], qsum[g][c], part);
                part += __shfl_xor_sync(0xffffffffu, part, 1);
                part += __shfl_xor_sync(0xffffffffu, part, 2);
                part += __shfl_xor_sync(0xffffffffu, part, 4);
                const float score = valid ? ks[u] * part : -INFINITY;
                float tmax = fmaxf(score, __shfl_xor_sync(0xffffffffu, score, 8));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
                if (tmax > m[g]) {  // warp-uniform: rescale what has been accumulated so far
                    const float corr = expf(m[g] - tmax);  // exp(-inf) = 0 on the first tile
                    l[g] *= corr, zacc[g] *= corr;
#pragma unroll
                    for (int i = 0; i < 16; ++i) acc[g][i] *= corr;
                    m[g] = tmax;
                }
                const float pr = valid ? expf(score - m[g]) : 0.0f;
                const float w = pr * vs[u];
                l[g] += pr;
                zacc[g] = fmaf(w, vz[u], zacc[g]);
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[g][i] = fmaf(w, vd[i], acc[g][i]);
            }
        }
    }

    // merge the four token lanes of the warp (same running max), then the warps through shared memory
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int o = 8; o <= 16; o <<= 1) {
            l[g] += __shfl_xor_sync(0xffffffffu, l[g], o);
            zacc[g] += __shfl_xor_sync(0xffffffffu, zacc[g], o);
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[g][i] += __shfl_xor_sync(0xffffffffu, acc[g][i], o);
        }
        if (j == 0) {
#pragma unroll
            for (int i = 0; i < 16; ++i) red[warp][g][16 * c + i] = acc[g][i] - zacc[g];  // zero-point term folded in
            if (c == 0) red[warp][g][kKvD] = m[g], red[warp][g][kKvD + 1] = l[g];
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * kKvPartial; i += blockDim.x) {
        const int g = i / kKvPartial, d = i % kKvPartial;
        float mm = -INFINITY;
        for (int w = 0; w < kKvWarps; ++w) mm = fmaxf(mm, red[w][g][kKvD]);
        float val;
        if (d == kKvD) {
            val = mm;
        } else {
            val = 0.0f;
            for (int w = 0; w < kKvWarps; ++w) {
                const float mw = red[w][g][kKvD];
                if (mw > -INFINITY) val = fmaf(red[w][g][d], expf(mw - mm), val);
            }
        }
        p.partial[(static_cast<size_t>(head0 + g) * p.splits + split) * kKvPartial + d] = val;
    }
}

// Merge the splits of each query head: one CTA per head, one thread per dimension.
__global__ void __launch_bounds__(kKvD)
kv4_attention_combine_kernel(const Kv4Params p) {
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.x, d = threadIdx.x;
    const float* base = p.partial + static_cast<size_t>(h) * p.splits * kKvPartial;
    float mm = -INFINITY;
    for (int s = 0; s < p.splits; ++s) mm = fmaxf(mm, base[s * kKvPartial + kKvD]);
    float num = 0.0f, den = 0.0f;
    for (int s = 0; s < p.splits; ++s) {
        const float ms = base[s * kKvPartial + kKvD];
        if (ms > -INFINITY) {
            const float f = expf(ms - mm);
            num = fmaf(base[s * kKvPartial + d], f, num);
            den = fmaf(base[s * kKvPartial + kKvD + 1], f, den);
        }
    }
    p.out[static_cast<size_t>(h) * kKvD + d] = num / den;
}

}  // namespace qift

// KV4: asymmetric 4-bit key / value cache (Sec. 4.1: "asymmetric key and value quantization with
// clipping ratios of 0.95") and the single-query decode attention that reads it.
//
// Cache layout (device memory, owned by the caller), head-major so that the tokens of one KV head are
// contiguous.  Keys: codes uint8 [Hkv][T_cap][D/2], two neighbouring dimensions of a token per byte
// (even dimension in the low nibble).  Values: codes uint8 [Hkv][T_cap/2][D], two consecutive tokens
// of a dimension per byte (even token in the low nibble).  Both: scale fp32 [Hkv][T_cap], zero fp32
// [Hkv][T_cap] (the integer zero-point 0..15 as a float).  T_cap is even.
// D = 128 (the head dimension of the LLaMA models the paper evaluates).
#pragma once

#include <cuda_fp16.h>

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
// Quantizes the vector whose four elements per lane are in v (rotating it first when had_block > 1);
// returns the lane's four codes in the low 16 bits (element e at bits 4e) and the vector's scale and
// zero-point.
__device__ __forceinline__ uint32_t kv4_quantize_vector(float (&v)[4], int lane, int had_block, float inv_sqrt_b, float clip, float& s,
                                                        float& z) {
    if (had_block > 1) {
        // element index = 4 * lane + e; strides below had_block only
        {
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
    s = 1.0f, z = 0.0f;
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
    return packed;
}

template <bool BF16_IN>
__device__ __forceinline__ void kv4_load_vector(const void* X, long long r, int lane, float (&v)[4]) {
    if constexpr (BF16_IN) {
        const uint2 w = reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(X) + r * kKvD)[lane];
        v[0] = __uint_as_float(w.x << 16), v[1] = __uint_as_float(w.x & 0xffff0000u);
        v[2] = __uint_as_float(w.y << 16), v[3] = __uint_as_float(w.y & 0xffff0000u);
    } else {
        const float4 f = reinterpret_cast<const float4*>(static_cast<const float*>(X) + r * kKvD)[lane];
        v[0] = f.x, v[1] = f.y, v[2] = f.z, v[3] = f.w;
    }
}

// Keys: one warp per (token, head); byte = two neighbouring dimensions.
template <bool BF16_IN>
__global__ void __launch_bounds__(256)
kv4_quantize_kernel(const void* __restrict__ X, long long rows, int H, int had_block, float inv_sqrt_b, float clip, int t0,
                    int T_cap, uint8_t* __restrict__ codes, float* __restrict__ scale, float* __restrict__ zero) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long r = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);  // input row = token * H + head
    if (r >= rows) return;
    float v[4], s, z;
    kv4_load_vector<BF16_IN>(X, r, lane, v);
    const uint32_t packed = kv4_quantize_vector(v, lane, had_block, inv_sqrt_b, clip, s, z);
    const long long t = r / H;
    const int h = static_cast<int>(r - t * H);
    const size_t slot = static_cast<size_t>(h) * T_cap + t0 + t;
    reinterpret_cast<uint16_t*>(codes + slot * kKvRowBytes)[lane] = static_cast<uint16_t>(packed);
    if (lane == 0) {
        scale[slot] = s;
        zero[slot] = z;
    }
}

// Values: one warp per (pair of consecutive cache slots, head); byte = the two tokens of the pair at one
// dimension (even slot in the low nibble), bytes [H][T_cap / 2][D].  A slot of the pair that is not
// among the T new tokens keeps its nibble (no other warp of the launch touches the pair).
template <bool BF16_IN>
__global__ void __launch_bounds__(256)
kv4_quantize_pairs_kernel(const void* __restrict__ X, int T, int H, int had_block, float inv_sqrt_b, float clip, int t0, int T_cap,
                          uint8_t* __restrict__ codes, float* __restrict__ scale, float* __restrict__ zero) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int first_pair = t0 >> 1, n_pairs = ((t0 + T + 1) >> 1) - first_pair;
    const long long w = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);  // (pair, head)
    if (w >= static_cast<long long>(n_pairs) * H) return;
    const int pair = first_pair + static_cast<int>(w / H), h = static_cast<int>(w % H);
    uint32_t nib[2] = {0, 0};
    bool have[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int slot = 2 * pair + k;
        have[k] = slot >= t0 && slot < t0 + T;
        if (have[k]) {  // warp-uniform
            float v[4], s, z;
            kv4_load_vector<BF16_IN>(X, static_cast<long long>(slot - t0) * H + h, lane, v);
            nib[k] = kv4_quantize_vector(v, lane, had_block, inv_sqrt_b, clip, s, z);
            if (lane == 0) {
                scale[static_cast<size_t>(h) * T_cap + slot] = s;
                zero[static_cast<size_t>(h) * T_cap + slot] = z;
            }
        }
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(codes + (static_cast<size_t>(h) * (T_cap >> 1) + pair) * kKvD) + lane;
    // spread the four codes of each token over four bytes: token k's code e -> byte e, nibble k
    uint32_t lo = (nib[0] & 0xf) | ((nib[0] & 0xf0) << 4) | ((nib[0] & 0xf00) << 8) | ((nib[0] & 0xf000) << 12);
    uint32_t hi = (nib[1] & 0xf) | ((nib[1] & 0xf0) << 4) | ((nib[1] & 0xf00) << 8) | ((nib[1] & 0xf000) << 12);
    uint32_t bytes = lo | (hi << 4);
    if (!(have[0] && have[1])) {
        const uint32_t old = *dst;
        bytes = have[0] ? (bytes & 0x0f0f0f0fu) | (old & 0xf0f0f0f0u) : (bytes & 0xf0f0f0f0u) | (old & 0x0f0f0f0fu);
    }
    *dst = bytes;
}

// ------------------------------------------------------------------------------------------------
// decode attention over the 4-bit cache (tensor cores)
// ------------------------------------------------------------------------------------------------
// out[h] = sum_t softmax_t(q[h] . Khat[t] / sqrt(D)) Vhat[t],  Khat = ks (kc - kz),  Vhat = vs (vc - vz),
// for the G = Hq / Hkv <= 8 query heads that share a KV head.
//
// Both products run on mma.sync.m16n8k16 (fp16 operands, fp32 accumulators) with the query heads as
// rows (rows g < 8: the high fp16 part of head g's operand, rows g + 8: its low part; heads beyond G are zero):
//   S[head][token] = sum_d q[head][d] * kc[token][d]          A = q,           B = key codes
//   O[head][d]    += sum_t w[head][t] * vc[t][d]              A = w = p * vs,  B = value codes
// The 4-bit codes are exact in fp16.  The fp32 operands q and w are each split into a high and a low
// fp16 part, which keeps the result at fp32 accuracy (the residual of the split is 2^-22 of the
// value); the two parts occupy rows g and g + 8 of the same instruction and their accumulators are
// added at the end, so the sixteen rows of the tile are all used.  Scales and zero-points stay out of the element path:
//   score = ks[t] * (S - kz[t] * sum_d q[d]),     O_final = O - sum_t w[t] * vz[t].
// A byte of the cache is exactly one operand register: two neighbouring dimensions of a token for the
// keys (the k index of the first product), two neighbouring tokens of a dimension for the values (the
// k index of the second), low nibble = lower index.  Which dimension sits at which k (or n) position
// of an instruction is free as long as both operands agree, and is chosen so that a lane reads 16
// contiguous bytes per cache row:
//   keys:   lane (g, cq) holds bytes [16cq, 16cq+16) of token g's row; k-step ks uses bytes 2ks, 2ks+1,
//           i.e. k positions 2cq, 2cq+1 <-> dimensions 32cq + 4ks, +1 and 2cq+8, 2cq+9 <-> 32cq + 4ks + 2, +3;
//   values: lane (g, cq) holds bytes [16g, 16g+16) of pair rows cq and cq+4; n-tile nt uses byte nt,
//           i.e. column g of n-tile nt <-> dimension 16g + nt.
// Grid (splits, Hkv): a CTA takes a contiguous range of tokens of one KV head, its four warps take
// 16-token tiles in turn, each with its own running max / denominator / numerator (merged through
// shared memory at the end, and across splits by kv4_attention_combine_kernel).
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

constexpr int kKvWarps = 4;
constexpr int kKvTile = 16;          // tokens per warp tile
constexpr int kKvPartial = kKvD + 2;
constexpr float kKvSlack = 8.0f;     // weights stay below e^8 relative to the reference point

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Byte `pos` of a word -> two fp16 codes (low nibble in the low half), three instructions: the byte is
// copied into both halves, its low nibble kept in the low half and its high nibble (in place, i.e.
// times 16) in the high half, each under the exponent of 1024: the halves read 1024 + c_lo and
// 1024 + 16 c_hi; one fused multiply-add by (1, 1/16) plus (-1024, -64) leaves (c_lo, c_hi), exactly.
__device__ __forceinline__ uint32_t byte_to_half2(uint32_t word, int pos) {
    const uint32_t x2 = __byte_perm(word, 0u, 0x4040u | static_cast<uint32_t>(pos) | (static_cast<uint32_t>(pos) << 8));
    const uint32_t h = (x2 & 0x00f0000fu) | 0x64006400u;
    uint32_t r;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(h), "r"(0x2c003c00u), "r"(0xd400e400u));
    return r;
}

// fp32 pair -> high fp16 parts and low fp16 parts (the residuals).
__device__ __forceinline__ void split_half2(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __half2 h = __floats2half2_rn(x, y);
    const float2 back = __half22float2(h);
    const __half2 l = __floats2half2_rn(x - back.x, y - back.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

__global__ void __launch_bounds__(32 * kKvWarps, 2)
kv4_attention_partial_kernel(const Kv4Params p) {
    __shared__ float red[kKvWarps][8][kKvPartial];
    pdl_launch_dependents();
    pdl_wait();
    const int kv = blockIdx.y, split = blockIdx.x, G = p.heads_per_kv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, cq = lane & 3;

    const int t_begin = split * p.tokens_per_split;
    const int t_end = min(p.T, t_begin + p.tokens_per_split);
    const size_t head_row = static_cast<size_t>(kv) * p.T_cap;
    const uint8_t* vbase = p.v_codes + static_cast<size_t>(kv) * (p.T_cap >> 1) * kKvD;
    const int last_row = p.T_cap - 1, last_pair = (p.T_cap >> 1) - 1;

    // loads of a tile: key rows of tokens tb+g and tb+8+g, value pair rows tb/2+cq and tb/2+4+cq, scales and
    // zero-points of this lane's four tokens tb + 8n + 2cq + {0,1}; issued one tile ahead of their use
    struct Tile {
        uint4 kraw[2], vraw[2];
        float2 ksc[2], kzp[2], vsc[2], vzp[2];
    };
    const uint8_t* kbase = p.k_codes + head_row * kKvRowBytes;
    const float* ksb = p.k_scale + head_row;
    const float* kzb = p.k_zero + head_row;
    const float* vsb = p.v_scale + head_row;
    const float* vzb = p.v_zero + head_row;
    const uint32_t klane = static_cast<uint32_t>(g) * kKvRowBytes + 16u * cq;
    const uint32_t vlane = static_cast<uint32_t>(cq) * kKvD + 16u * g;
    // clamped 32-bit byte offsets from per-head base pointers: rows past the end of the arrays (a last tile
    // that crosses T_cap) read the last row instead; offsets grow with the row, so one min per load does it
    const uint32_t kmax = static_cast<uint32_t>(last_row) * kKvRowBytes + 16u * cq;
    const uint32_t vmax = static_cast<uint32_t>(last_pair) * kKvD + 16u * g;
    const uint32_t smax = static_cast<uint32_t>(last_row - 1);
    auto load_tile = [&](Tile& x, int tb) {
        const uint32_t koff = static_cast<uint32_t>(tb) * kKvRowBytes + klane;
        const uint32_t voff = static_cast<uint32_t>(tb >> 1) * kKvD + vlane;
        const uint32_t so = static_cast<uint32_t>(tb) + 2u * cq;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            x.kraw[n] = *reinterpret_cast<const uint4*>(kbase + min(koff + n * 8u * kKvRowBytes, kmax));
            x.vraw[n] = *reinterpret_cast<const uint4*>(vbase + min(voff + n * 4u * kKvD, vmax));
            const uint32_t t = min(so + n * 8u, smax);   // even: the pair t, t+1 is inside the arrays
            x.ksc[n] = *reinterpret_cast<const float2*>(ksb + t);
            x.kzp[n] = *reinterpret_cast<const float2*>(kzb + t);
            x.vsc[n] = *reinterpret_cast<const float2*>(vsb + t);
            x.vzp[n] = *reinterpret_cast<const float2*>(vzb + t);
        }
    };
    // the warp's first tile is requested before the query is touched: the two latencies overlap
    constexpr int kTileStride = kKvTile * kKvWarps;
    Tile ta, tb2;
    int tb = t_begin + kKvTile * warp;
    if (tb < t_end) load_tile(ta, tb);

    // query fragments: row g (head kv*G + g, zero beyond G), scaled by 1/sqrt(D), split in two fp16 parts
    uint32_t qh[8][2], ql[8][2];
    float qsum = 0.0f;  // sum over all dimensions of (high + low) parts of head g
    {
        const float* qrow = p.q + static_cast<size_t>(kv * G + (g < G ? g : 0)) * kKvD;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            float4 f = *reinterpret_cast<const float4*>(qrow + 32 * cq + 4 * ks);
            if (g >= G) f = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            f.x = __fmul_rn(f.x, p.inv_sqrt_d), f.y = __fmul_rn(f.y, p.inv_sqrt_d);
            f.z = __fmul_rn(f.z, p.inv_sqrt_d), f.w = __fmul_rn(f.w, p.inv_sqrt_d);
            split_half2(f.x, f.y, qh[ks][0], ql[ks][0]);
            split_half2(f.z, f.w, qh[ks][1], ql[ks][1]);
            qsum += (f.x + f.y) + (f.z + f.w);
        }
        qsum += __shfl_xor_sync(0xffffffffu, qsum, 1);
        qsum += __shfl_xor_sync(0xffffffffu, qsum, 2);
    }

    float o[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[nt][i] = 0.0f;
    float m_run = -INFINITY, l_run = 0.0f, z_run = 0.0f;  // of head g (l and z: this lane's tokens only)

    auto process_tile = [&](const Tile& cur, int tb) {
        const uint4(&kraw)[2] = cur.kraw;
        const uint4(&vraw)[2] = cur.vraw;
        const float2(&ksc)[2] = cur.ksc;
        const float2(&kzp)[2] = cur.kzp;
        const float2(&vsc)[2] = cur.vsc;
        const float2(&vzp)[2] = cur.vzp;
        // ---- S = q . codes for the two 8-token n-tiles
        float sc[2][4];
#pragma unroll
        for (int n = 0; n < 2; ++n) {
#pragma unroll
            for (int i = 0; i < 4; ++i) sc[n][i] = 0.0f;
            const uint32_t w[4] = {kraw[n].x, kraw[n].y, kraw[n].z, kraw[n].w};
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t b0 = byte_to_half2(w[ks >> 1], 2 * (ks & 1)), b1 = byte_to_half2(w[ks >> 1], 2 * (ks & 1) + 1);
                mma_f16(sc[n], qh[ks][0], ql[ks][0], qh[ks][1], ql[ks][1], b0, b1);  // rows g: high parts, rows g+8: low parts
            }
        }
        // ---- scores of head g for this lane's four tokens, running max, weights
        float s4[4];
        float tmax = -INFINITY;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            const int t = tb + 8 * n + 2 * cq;
            s4[2 * n] = (t < t_end) ? ksc[n].x * fmaf(-kzp[n].x, qsum, sc[n][0] + sc[n][2]) : -INFINITY;
            s4[2 * n + 1] = (t + 1 < t_end) ? ksc[n].y * fmaf(-kzp[n].y, qsum, sc[n][1] + sc[n][3]) : -INFINITY;
            tmax = fmaxf(tmax, fmaxf(s4[2 * n], s4[2 * n + 1]));
        }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        // The reference point of the exponentials only has to keep them in range: it is moved (and the
        // accumulators rescaled) when a row's scores exceed it by more than kKvSlack, not at every new max.
        const bool grew = tmax > m_run + kKvSlack;
        if (__any_sync(0xffffffffu, grew)) {
            const float corr = grew ? expf(m_run - tmax) : 1.0f;  // exp(-inf) = 0 on a row's first tile
            l_run *= corr, z_run *= corr;
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) o[nt][0] *= corr, o[nt][1] *= corr, o[nt][2] *= corr, o[nt][3] *= corr;
            if (grew) m_run = tmax;
        }
        float w4[4];
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            // slots past the split's end may hold anything (a cache is filled as tokens arrive), NaN included:
            // their scale and zero-point are replaced, not multiplied by a zero weight
            const bool in0 = s4[2 * n] > -INFINITY, in1 = s4[2 * n + 1] > -INFINITY;
            const float p0 = in0 ? expf(s4[2 * n] - m_run) : 0.0f;
            const float p1 = in1 ? expf(s4[2 * n + 1] - m_run) : 0.0f;
            l_run += p0 + p1;
            w4[2 * n] = in0 ? p0 * vsc[n].x : 0.0f, w4[2 * n + 1] = in1 ? p1 * vsc[n].y : 0.0f;
            z_run = fmaf(w4[2 * n], in0 ? vzp[n].x : 0.0f, fmaf(w4[2 * n + 1], in1 ? vzp[n].y : 0.0f, z_run));
        }
        // ---- O += w . value codes: k = the tile's 16 tokens, A rows = heads
        uint32_t wh[2], wl[2];
        split_half2(w4[0], w4[1], wh[0], wl[0]);
        split_half2(w4[2], w4[3], wh[1], wl[1]);
        const uint32_t va[4] = {vraw[0].x, vraw[0].y, vraw[0].z, vraw[0].w};
        const uint32_t vb[4] = {vraw[1].x, vraw[1].y, vraw[1].z, vraw[1].w};
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            const uint32_t b0 = byte_to_half2(va[nt >> 2], nt & 3), b1 = byte_to_half2(vb[nt >> 2], nt & 3);
            mma_f16(o[nt], wh[0], wl[0], wh[1], wl[1], b0, b1);
        }
    };
    // two tile buffers used alternately, each loaded one tile ahead of its use
    {
        constexpr int stride = kTileStride;
        while (tb < t_end) {
            if (tb + stride < t_end) load_tile(tb2, tb + stride);
            process_tile(ta, tb);
            tb += stride;
            if (tb >= t_end) break;
            if (tb + stride < t_end) load_tile(ta, tb + stride);
            process_tile(tb2, tb);
            tb += stride;
        }
    }

    // ---- merge: the four lanes of a row, then the warps through shared memory
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1), l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    z_run += __shfl_xor_sync(0xffffffffu, z_run, 1), z_run += __shfl_xor_sync(0xffffffffu, z_run, 2);
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {  // column 2cq + e of n-tile nt is dimension 16 (2cq + e) + nt
        red[warp][g][16 * (2 * cq) + nt] = (o[nt][0] + o[nt][2]) - z_run;
        red[warp][g][16 * (2 * cq + 1) + nt] = (o[nt][1] + o[nt][3]) - z_run;
    }
    if (cq == 0) red[warp][g][kKvD] = m_run, red[warp][g][kKvD + 1] = l_run;
    __syncthreads();
    for (int i = threadIdx.x; i < G * kKvPartial; i += blockDim.x) {
        const int h = i / kKvPartial, d = i % kKvPartial;
        float mm = -INFINITY;
        for (int w = 0; w < kKvWarps; ++w) mm = fmaxf(mm, red[w][h][kKvD]);
        float val;
        if (d == kKvD) {
            val = mm;
        } else {
            val = 0.0f;
            for (int w = 0; w < kKvWarps; ++w) {
                const float mw = red[w][h][kKvD];
                if (mw > -INFINITY) val = fmaf(red[w][h][d], expf(mw - mm), val);
            }
        }
        p.partial[(static_cast<size_t>(kv * G + h) * p.splits + split) * kKvPartial + d] = val;
    }
}

// Merge the splits of each query head: one CTA per head, four groups of 64 threads.  Group r takes splits
// r, r+4, ...; a thread takes two neighbouring dimensions.  The numerators of a group's first splits are
// requested before the weights exp(m_s - max) exist (one exponential per split, computed by thread s), so the
// kernel spends one round trip to memory on them instead of one per split; the groups meet in shared memory.
constexpr int kKvMaxSplits = 1024;
constexpr int kKvCombineThreads = 256;
constexpr int kKvCombineGroups = kKvCombineThreads / (kKvD / 2);
constexpr int kKvCombineAhead = 8;  // splits per group whose loads are issued up front (32 splits in all)
__global__ void __launch_bounds__(kKvCombineThreads)
kv4_attention_combine_kernel(const Kv4Params p) {
    __shared__ float weight[kKvMaxSplits];
    __shared__ float wmax[kKvCombineThreads / 32];
    __shared__ float2 gnum[kKvCombineGroups][kKvD / 2];
    __shared__ float gden[kKvCombineGroups];
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.x, tid = threadIdx.x;
    const int grp = tid / (kKvD / 2), j = tid % (kKvD / 2);
    const float* base = p.partial + static_cast<size_t>(h) * p.splits * kKvPartial;
    float2 pre[kKvCombineAhead];
    float dpre[kKvCombineAhead];
#pragma unroll
    for (int i = 0; i < kKvCombineAhead; ++i) {
        const int s = grp + kKvCombineGroups * i;
        pre[i] = make_float2(0.0f, 0.0f), dpre[i] = 0.0f;
        if (s < p.splits) {
            pre[i] = *reinterpret_cast<const float2*>(base + static_cast<size_t>(s) * kKvPartial + 2 * j);
            dpre[i] = base[static_cast<size_t>(s) * kKvPartial + kKvD + 1];
        }
    }
    float msv[kKvMaxSplits / kKvCombineThreads];
    float mm = -INFINITY;
#pragma unroll
    for (int i = 0; i < kKvMaxSplits / kKvCombineThreads; ++i) {
        const int s = tid + kKvCombineThreads * i;
        msv[i] = (s < p.splits) ? base[static_cast<size_t>(s) * kKvPartial + kKvD] : -INFINITY;
        mm = fmaxf(mm, msv[i]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
    if ((tid & 31) == 0) wmax[tid >> 5] = mm;
    __syncthreads();
    mm = wmax[0];
#pragma unroll
    for (int w = 1; w < kKvCombineThreads / 32; ++w) mm = fmaxf(mm, wmax[w]);
#pragma unroll
    for (int i = 0; i < kKvMaxSplits / kKvCombineThreads; ++i) {
        const int s = tid + kKvCombineThreads * i;
        if (s < p.splits) weight[s] = (msv[i] > -INFINITY) ? expf(msv[i] - mm) : 0.0f;
    }
    __syncthreads();
    float2 num = make_float2(0.0f, 0.0f);
    float den = 0.0f;
#pragma unroll
    for (int i = 0; i < kKvCombineAhead; ++i) {
        const int s = grp + kKvCombineGroups * i;
        if (s < p.splits) {
            const float f = weight[s];
            num.x = fmaf(pre[i].x, f, num.x), num.y = fmaf(pre[i].y, f, num.y);
            den = fmaf(dpre[i], f, den);
        }
    }
    for (int s = grp + kKvCombineGroups * kKvCombineAhead; s < p.splits; s += kKvCombineGroups) {
        const float f = weight[s];
        const float2 v = *reinterpret_cast<const float2*>(base + static_cast<size_t>(s) * kKvPartial + 2 * j);
        num.x = fmaf(v.x, f, num.x), num.y = fmaf(v.y, f, num.y);
        den = fmaf(base[static_cast<size_t>(s) * kKvPartial + kKvD + 1], f, den);
    }
    gnum[grp][j] = num;
    if (j == 0) gden[grp] = den;
    __syncthreads();
    if (tid < kKvD / 2) {
        float2 n = gnum[0][tid];
        float d = gden[0];
#pragma unroll
        for (int r = 1; r < kKvCombineGroups; ++r) n.x += gnum[r][tid].x, n.y += gnum[r][tid].y, d += gden[r];
        *reinterpret_cast<float2*>(p.out + static_cast<size_t>(h) * kKvD + 2 * tid) = make_float2(n.x / d, n.y / d);
    }
}

}  // namespace qift

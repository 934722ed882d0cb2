// Blockwise Walsh-Hadamard rotation, fused per-token INT4 activation quantizer, offline rotation.
//
// One CTA per row.  The row lives in shared memory as fp32 (padded, see pad_index); the butterfly runs in radix-16 passes
// (four stages per pass in registers), stages in ascending stride so that every add/sub sees the
// same operands as the textbook in-place butterfly -- the result is then bit-identical to it
// whatever the thread mapping, because each stage is a set of independent IEEE additions.
#pragma once

#include "common.cuh"

namespace qift {

constexpr int kRowThreads = 256;
// Threads per row CTA: the shared-memory passes give each thread 32 elements, so rows up to 4096
// keep every thread busy with 128.
inline int row_threads(int K) { return K <= 4096 ? 128 : kRowThreads; }
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

// Two fp32 values in one 64-bit register, operated on by the packed fp32 instructions of sm_100
// (one issue slot for two IEEE round-to-nearest operations, each identical to its scalar form).
typedef unsigned long long f32x2_t;
__device__ __forceinline__ f32x2_t f2_make(float lo, float hi) {
    f32x2_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_split(f32x2_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2_t f2_add(f32x2_t a, f32x2_t b) {
    f32x2_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2_t f2_sub(f32x2_t a, f32x2_t b) {
    f32x2_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2_t f2_mul(f32x2_t a, f32x2_t b) {
    f32x2_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2_t f2_fma(f32x2_t a, f32x2_t b, f32x2_t c) {
    f32x2_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// The same butterfly on R column pairs: v[i] holds the two neighbouring columns of group element i.
template <int R>
__device__ __forceinline__ void butterfly_pairs(f32x2_t (&v)[R], int active_stages) {
#pragma unroll
    for (int s = 0, h = 1; h < R; h <<= 1, ++s) {
        if (s < active_stages) {
#pragma unroll
            for (int i = 0; i < R; ++i) {
                if ((i & h) == 0) {
                    const f32x2_t a = v[i], b = v[i + h];
                    v[i] = f2_add(a, b);
                    v[i + h] = f2_sub(a, b);
                }
            }
        }
    }
}

__device__ __forceinline__ float max_abs2(f32x2_t v, float m) {
    float lo, hi;
    f2_split(v, lo, hi);
    return fmaxf(m, fmaxf(fabsf(lo), fabsf(hi)));
}

// Shared-memory row layout.  Element e lives at pad_index(e): four floats of padding after every 32
// and sixteen more after every 256.  With it every access pattern of the kernels below is free of
// bank conflicts: 64 contiguous bytes per lane (first pass, quantizer), 16 lanes x stride-16 groups
// of two neighbouring 256-blocks (second pass), consecutive lanes at strides >= 256 (later passes);
// and the offsets between the elements of one butterfly group are compile-time constants.
__host__ __device__ constexpr int pad_index(int e) { return e + ((e >> 5) << 2) + ((e >> 8) << 4); }
__host__ __device__ inline size_t padded_row_bytes(int K) { return static_cast<size_t>(pad_index(K)) * 4; }

// One radix-16 pass over the row in shared memory: strides SB, 2SB, 4SB, 8SB (those below B).
// A thread takes two neighbouring columns of a group (64-bit accesses, packed arithmetic).
// Returns the thread's running max |value| of what it wrote when WANT_MAX.
template <int SB, bool WANT_MAX>
__device__ __forceinline__ float wht_pass_smem(float* row, int K, int B) {
    constexpr int LSB = (SB == 16) ? 4 : (SB == 256) ? 8 : 12;
    const int stages = min(4, (31 - __clz(B)) - LSB);  // B is a power of two above SB
    const int R = 1 << stages;                         // elements of one group
    const int pair_groups = K >> (stages + 1);
    float amax = 0.0f;
    if (stages == 4) {
        for (int q = threadIdx.x; q < pair_groups; q += blockDim.x) {
            float* base = row + pad_index(((q >> (LSB - 1)) << (LSB + 4)) + 2 * (q & (SB / 2 - 1)));
            f32x2_t v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j)
                v[j] = *reinterpret_cast<const f32x2_t*>(base + (SB == 16 ? 16 * j + 4 * (j >> 1) : j * pad_index(SB)));
            butterfly_pairs<16>(v, 4);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (WANT_MAX) amax = max_abs2(v[j], amax);
                *reinterpret_cast<f32x2_t*>(base + (SB == 16 ? 16 * j + 4 * (j >> 1) : j * pad_index(SB))) = v[j];
            }
        }
    } else {  // last, partial pass: 2, 4 or 8 elements per group
        for (int q = threadIdx.x; q < pair_groups; q += blockDim.x) {
            const int e0 = ((q >> (LSB - 1)) << (LSB + stages)) + 2 * (q & (SB / 2 - 1));
            f32x2_t v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (j < R) ? *reinterpret_cast<const f32x2_t*>(row + pad_index(e0 + j * SB)) : 0ull;
            butterfly_pairs<8>(v, stages);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < R) {
                    *reinterpret_cast<f32x2_t*>(row + pad_index(e0 + j * SB)) = v[j];
                    if (WANT_MAX) amax = max_abs2(v[j], amax);
                }
        }
    }
    return amax;
}

// Hadamard matrix of order 28 (there is no Sylvester matrix of that order): Paley's second construction
// with q = 13.  chi = quadratic character mod 13; conference matrix C = [0 1; 1 Q] with Q[i][j] =
// chi(i - j); H = [C + I, C - I; C - I, -C - I].  Built at compile time, so that the fully unrolled
// 28-point transform below turns every entry into the sign of an add.
struct Hadamard28 {
    signed char v[28][28];
};
constexpr Hadamard28 make_hadamard28() {
    Hadamard28 t{};
    int chi[13] = {};
    for (int a = 1; a < 13; ++a) chi[a] = -1;
    for (int x = 1; x < 13; ++x) chi[(x * x) % 13] = 1;
    for (int i = 0; i < 14; ++i)
        for (int j = 0; j < 14; ++j) {
            const int c = (i == 0 || j == 0) ? ((i == j) ? 0 : 1) : chi[((i - j) % 13 + 13) % 13];
            const int d = (i == j) ? 1 : 0;
            t.v[i][j] = static_cast<signed char>(c + d);
            t.v[i][j + 14] = static_cast<signed char>(c - d);
            t.v[i + 14][j] = static_cast<signed char>(c - d);
            t.v[i + 14][j + 14] = static_cast<signed char>(-c - d);
        }
    return t;
}
constexpr Hadamard28 kH28 = make_hadamard28();

template <int R, int J>
__device__ __forceinline__ float h28_acc(const float (&x)[28], float acc) {  // terms J..27 of row R, in order
    if constexpr (J < 28) {
        constexpr bool plus = kH28.v[R][J] > 0;
        return h28_acc<R, J + 1>(x, plus ? __fadd_rn(acc, x[J]) : __fsub_rn(acc, x[J]));
    } else {
        return acc;
    }
}
template <int R>
__device__ __forceinline__ float h28_row(const float (&x)[28]) {  // signed sum in ascending order, first term +-x[0]
    constexpr bool plus0 = kH28.v[R][0] > 0;
    return h28_acc<R, 1>(x, plus0 ? x[0] : -x[0]);
}
template <int R>
__device__ __forceinline__ void h28_rows(const float (&x)[28], float (&y)[28]) {
    if constexpr (R < 28) {
        y[R] = h28_row<R>(x);
        h28_rows<R + 1>(x, y);
    }
}

// Second factor of the full-dimension rotation H_28 (x) H_P of a row of K = 28 P entries (the first, the
// Sylvester transform of every block of P, has been done): H_28 across the 28 blocks at every position.
// Returns the thread's max |value| written.
__device__ __forceinline__ float kron28_pass_smem(float* row, int P) {
    float amax = 0.0f;
    for (int i = threadIdx.x; i < P; i += blockDim.x) {
        float x[28], y[28];
#pragma unroll
        for (int j = 0; j < 28; ++j) x[j] = row[pad_index(j * P + i)];
        h28_rows<0>(x, y);
#pragma unroll
        for (int j = 0; j < 28; ++j) {
            row[pad_index(j * P + i)] = y[j];
            amax = fmaxf(amax, fabsf(y[j]));
        }
    }
    return amax;
}

// Loads the row (fp32 or bf16), runs the strides 1..8 in registers, leaves the row in shared memory
// (padded layout), then finishes the transform there.  B <= 1 means no rotation.  Returns the
// thread's partial max |value| of the transformed row (taken in whichever pass ran last).
// KRON: compiled with the 28-point pass (56 more registers); kernels without it reject nothing -- the host
// picks the variant from had_block.
template <bool BF16_IN, bool KRON = false>
__device__ __forceinline__ float load_and_transform(const void* X, size_t row_index, int K, int had_block, float* row) {
    // had_block: a power of two = block-diagonal Sylvester blocks; K = 28 * 2^p = the full-dimension rotation
    const bool kron = KRON && (had_block & (had_block - 1)) != 0;
    const int B = kron ? K / 28 : had_block;
    const int groups = K / 16;
    const int stages0 = (B > 1) ? min(4, 31 - __clz(B)) : 0;
    float amax = 0.0f;
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
        f32x2_t pr[8];  // stride 1 on scalars, strides 2, 4, 8 on pairs of neighbours
        if (stages0 == 4) {  // the usual case, without per-stage tests
#pragma unroll
            for (int i = 0; i < 8; ++i) pr[i] = f2_make(__fadd_rn(v[2 * i], v[2 * i + 1]), __fsub_rn(v[2 * i], v[2 * i + 1]));
            butterfly_pairs<8>(pr, 3);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                pr[i] = (stages0 > 0) ? f2_make(__fadd_rn(v[2 * i], v[2 * i + 1]), __fsub_rn(v[2 * i], v[2 * i + 1]))
                                      : f2_make(v[2 * i], v[2 * i + 1]);
            butterfly_pairs<8>(pr, stages0 - 1);
        }
        if (B <= 16) {
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = max_abs2(pr[i], amax);
        }
        ulonglong2* dst = reinterpret_cast<ulonglong2*>(row + pad_index(16 * q));
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_ulonglong2(pr[2 * i], pr[2 * i + 1]);
    }
    __syncthreads();
    if (B > 16) {
        amax = (B <= 256) ? wht_pass_smem<16, true>(row, K, B) : wht_pass_smem<16, false>(row, K, B);
        __syncthreads();
    }
    if (B > 256) {
        amax = (B <= 4096) ? wht_pass_smem<256, true>(row, K, B) : wht_pass_smem<256, false>(row, K, B);
        __syncthreads();
    }
    if (B > 4096) {
        amax = wht_pass_smem<4096, true>(row, K, B);
        __syncthreads();
    }
    if constexpr (KRON) {
        if (kron) {
            amax = kron28_pass_smem(row, B);
            __syncthreads();
        }
    }
    return amax;
}

// Unit scale of a row from the threads' partial max |value|: s_u = (amax * clip) / 7 (1 for an all-
// zero row), and its reciprocal when that is a normal number (else 0: the quantizer then divides).
// The block-wide max and the two divisions are done by warp 0 alone and broadcast through shared
// memory, so the other warps spend no issue slots on them.  red: 10 floats.  Two barriers.
struct RowScale {
    float s_u, inv;
};
__device__ __forceinline__ RowScale block_row_scale(float v, float clip, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) red[warp] = v;
    __syncthreads();
    if (warp == 0) {
        float r = (lane < static_cast<int>(blockDim.x >> 5)) ? red[lane] : 0.0f;
#pragma unroll
        for (int o = kRowThreads / 64; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, o));
        if (lane == 0) {
            float s_u = 1.0f;
            if (r != 0.0f) s_u = __fdiv_rn(__fmul_rn(r, clip), 7.0f);
            const bool fast = (s_u >= 1e-30f) && (s_u <= 1e30f);
            red[8] = s_u;
            red[9] = fast ? __fdiv_rn(1.0f, s_u) : 0.0f;
        }
    }
    __syncthreads();
    return RowScale{red[8], red[9]};
}

// The quantizer computes clamp(rint(u / s_u), -8, 7), bit-identical to the IEEE division followed by
// round-half-even, without dividing: t = u * (1/s_u) differs from the correctly rounded quotient by less than
// 2^-19 wherever |t| <= 8, so unless t lies within 2^-17 of a rounding tie (k + 0.5) both round to
// the same integer; near a tie the exact quotient decides.  Clamping before rounding equals
// clamping after it (both are monotone and the bounds are integers).  Rounding is done by adding
// and subtracting 1.5 * 2^23.  Used while 1/s_u is a normal number; otherwise every element takes the exact quotient.
constexpr float kRoundMagic = 12582912.0f;
constexpr float kTieGuard = 0.49999237f;  // 0.5 - 2^-17
__device__ __forceinline__ float quantize_round_exact(float u, float s_u) {
    return fminf(fmaxf(rintf(__fdiv_rn(u, s_u)), -8.0f), 7.0f);
}
// Low byte of (r * mult + 1.5 * 2^23) is the two's-complement byte of the integer r * mult.
__device__ __forceinline__ uint32_t pack4_scaled(f32x2_t r01, f32x2_t r23, f32x2_t mult2) {
    const f32x2_t magic2 = f2_make(kRoundMagic, kRoundMagic);
    float b0, b1, b2, b3;
    f2_split(f2_fma(r01, mult2, magic2), b0, b1);
    f2_split(f2_fma(r23, mult2, magic2), b2, b3);
    return __byte_perm(__byte_perm(__float_as_uint(b0), __float_as_uint(b1), 0x0040),
                       __byte_perm(__float_as_uint(b2), __float_as_uint(b3), 0x0040), 0x5410);
}

// Quantizes the transformed row in shared memory with unit scale s_u and writes 16 bytes per group.
// mult_even / mult_odd: factor applied to the bytes of even / odd 32-bit words of each 16-byte group
// (1 and 1 for the public layout).  With WANT_SUM returns the thread's partial sum of the quantized
// values (taken from the packed bytes with dp4a, the factors divided out exactly).
// Where the 16-byte groups of a quantized row go.  RowMajorDst: group q at byte 16 q of the row.
struct RowMajorDst {
    int8_t* q_row;
    __device__ __forceinline__ void store(int q, uint4 v) const { reinterpret_cast<uint4*>(q_row)[q] = v; }
};

template <bool WANT_SUM, typename Dst>
__device__ __forceinline__ int quantize_row(const float* row, int K, RowScale sc, Dst dst, float mult_even, float mult_odd) {
    const int groups = K / 16;
    const float s_u = sc.s_u, inv = sc.inv;
    const bool fast = inv != 0.0f;
    const f32x2_t inv2 = f2_make(inv, inv), magic2 = f2_make(kRoundMagic, kRoundMagic);
    const f32x2_t me2 = f2_make(mult_even, mult_even), mo2 = f2_make(mult_odd, mult_odd);
    int sum_even = 0, sum_odd = 0;
    for (int q = threadIdx.x; q < groups; q += blockDim.x) {
        const ulonglong2* src = reinterpret_cast<const ulonglong2*>(row + pad_index(16 * q));
        f32x2_t r[8];
        float dmax = 0.0f;
        if (fast) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const ulonglong2 f = src[i];
                const f32x2_t e2[2] = {f.x, f.y};
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    float t0, t1;
                    f2_split(f2_mul(e2[j], inv2), t0, t1);
                    const f32x2_t t2 = f2_make(fminf(fmaxf(t0, -8.0f), 7.0f), fminf(fmaxf(t1, -8.0f), 7.0f));
                    r[2 * i + j] = f2_sub(f2_add(t2, magic2), magic2);
                    dmax = max_abs2(f2_sub(t2, r[2 * i + j]), dmax);
                }
            }
        }
        if (!fast || dmax > kTieGuard) {  // some element of the group is near a tie (rare): exact quotients for the group
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 f = *reinterpret_cast<const float4*>(&src[i]);
                r[2 * i] = f2_make(quantize_round_exact(f.x, s_u), quantize_round_exact(f.y, s_u));
                r[2 * i + 1] = f2_make(quantize_round_exact(f.z, s_u), quantize_round_exact(f.w, s_u));
            }
        }
        uint32_t out[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = pack4_scaled(r[2 * i], r[2 * i + 1], (i & 1) ? mo2 : me2);
        if (WANT_SUM) {
            sum_even = __dp4a(static_cast<int>(out[0]), 0x01010101, __dp4a(static_cast<int>(out[2]), 0x01010101, sum_even));
            sum_odd = __dp4a(static_cast<int>(out[1]), 0x01010101, __dp4a(static_cast<int>(out[3]), 0x01010101, sum_odd));
        }
        dst.store(q, make_uint4(out[0], out[1], out[2], out[3]));
    }
    return sum_even / static_cast<int>(mult_even) + sum_odd / static_cast<int>(mult_odd);
}

// K2: rotate + quantize one token row per CTA.
template <bool BF16_IN, bool KRON = false>
__global__ void __launch_bounds__(kRowThreads)
quantize_act_kernel(const void* __restrict__ X, int K, int B, float clip, float inv_sqrt_b,
                    int8_t* __restrict__ q_a, float* __restrict__ s_a) {
    extern __shared__ __align__(16) float row[];
    __shared__ float red[kRowThreads / 32 + 2];
    pdl_launch_dependents();
    pdl_wait();
    const size_t m = blockIdx.x;
    const RowScale sc = block_row_scale(load_and_transform<BF16_IN, KRON>(X, m, K, B, row), clip, red);
    if (threadIdx.x == 0) s_a[m] = (B > 1) ? __fmul_rn(sc.s_u, inv_sqrt_b) : sc.s_u;
    quantize_row<false>(row, K, sc, RowMajorDst{q_a + m * K}, 1.0f, 1.0f);
}

// S0: orthonormal blockwise rotation of fp32 rows.
template <bool KRON>
__global__ void __launch_bounds__(kRowThreads)
rotate_rows_kernel(const float* __restrict__ X, int K, int B, float inv_sqrt_b, float* __restrict__ Y) {
    extern __shared__ __align__(16) float row[];
    pdl_launch_dependents();
    pdl_wait();
    const size_t m = blockIdx.x;
    load_and_transform<false, KRON>(X, m, K, B, row);
    for (int i = threadIdx.x; i < K / 4; i += blockDim.x) {
        float4 f = *reinterpret_cast<const float4*>(row + pad_index(4 * i));
        f.x = __fmul_rn(f.x, inv_sqrt_b), f.y = __fmul_rn(f.y, inv_sqrt_b);
        f.z = __fmul_rn(f.z, inv_sqrt_b), f.w = __fmul_rn(f.w, inv_sqrt_b);
        reinterpret_cast<float4*>(Y + m * K)[i] = f;
    }
}

}  // namespace qift

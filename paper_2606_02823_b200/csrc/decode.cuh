// Decode-path product kernels (M <= 16): stream the packed codes from HBM once, decode in
// registers, accumulate exactly in INT32, apply the scales in the epilogue.
//
//  * linear_generic_kernel: one warp per output channel, dp4a.  Any M, any K; the slow, simple route.
//  * linear_decode_kernel:  the bandwidth route.  A producer warp stages 16-row x 128-word tiles of
//    packed weights (8 KB each, contiguous in memory: one cp.async.bulk per tile), and the matching
//    slice of q_a, into a shared-memory ring guarded by mbarriers.  The weight copies are issued BEFORE the programmatic-dependent-launch
//    wait, so in a stream of such launches the next layer's weights are in flight while the previous
//    layer finishes.  Eight consumer warps split each slab along K; a lane turns a packed word into
//    four u8 operand registers with one LOP3 each (w & (0x03030303 << 2t) = code * 4^t, which the
//    integer tensor-core instruction mma.sync.m16n8k32.u8.s8 multiplies against q_a directly) and keeps
//    one accumulator set per t; the exact division by 4^t, the affine level map
//    (level = alpha*code + gamma  =>  acc = alpha * sum code*q + gamma * sum q) and the scales come last.
#pragma once

#include "common.cuh"

namespace qift {

// ------------------------------------------------------------------------------------------------
// affine level maps:  acc = combine(S, Sb1, Sq)
//   S   = sum_k code * q        (INT4: code' = nibble ^ 8)
//   Sb1 = sum_k bit1(code) * q  (POT only)
//   Sq  = sum_k q
// ------------------------------------------------------------------------------------------------
template <int LV>
__device__ __forceinline__ int combine_generic(int S, int Sb1, int Sq) {
    if constexpr (LV == QIFT_LEVELS_MNZ) return 2 * S - 3 * Sq;
    if constexpr (LV == QIFT_LEVELS_SYM) return S - 2 * Sq;
    if constexpr (LV == QIFT_LEVELS_POT) return 3 * S - Sb1 - 4 * Sq;  // value+4 = 3c - b1
    return S - 8 * Sq;
}

constexpr int kGenericWarps = 8;
constexpr int kGenericTokens = 4;

template <int LV>
__global__ void __launch_bounds__(kGenericWarps * 32)
linear_generic_kernel(const uint32_t* __restrict__ packed, const float* __restrict__ s_n,
                      const int8_t* __restrict__ q_a, const float* __restrict__ s_a, int M, int N, int K,
                      void* __restrict__ Y, int y_bf16, int32_t* __restrict__ acc_debug) {
    constexpr int PER = codes_per_word(LV);
    constexpr int NPL = PER / 4;  // byte-lane groups per word
    constexpr int BITS = 32 / PER;
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * kGenericWarps + (threadIdx.x >> 5);
    if (n >= N) return;
    const int words = K / PER;
    const int pitch = round_up16(words);
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(q_a);
    const size_t qpitch = K / 4;
    for (int m0 = 0; m0 < M; m0 += kGenericTokens) {
        int S[kGenericTokens] = {}, Sb[kGenericTokens] = {}, Sq[kGenericTokens] = {};
        for (int j = lane; j < words; j += 32) {
            const uint32_t w = packed[packed_word_address(n, j, pitch)];
#pragma unroll
            for (int t = 0; t < NPL; ++t) {
                uint32_t a, hb = 0;
                if constexpr (LV == QIFT_LEVELS_INT4) {
                    a = ((w >> (BITS * t)) & 0x0f0f0f0fu) ^ 0x08080808u;
                } else {
                    a = (w >> (BITS * t)) & 0x03030303u;
                    hb = (a >> 1) & 0x01010101u;
                }
#pragma unroll
                for (int mm = 0; mm < kGenericTokens; ++mm) {
                    if (m0 + mm < M) {
                        const uint32_t qv = q32[(m0 + mm) * qpitch + static_cast<size_t>(j) * NPL + t];
                        S[mm] = dp4a_us(a, qv, S[mm]);
                        if constexpr (LV == QIFT_LEVELS_POT) Sb[mm] = dp4a_us(hb, qv, Sb[mm]);
                        Sq[mm] = dp4a_us(0x01010101u, qv, Sq[mm]);
                    }
                }
            }
        }
#pragma unroll
        for (int mm = 0; mm < kGenericTokens; ++mm) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                S[mm] += __shfl_xor_sync(0xffffffffu, S[mm], o);
                Sb[mm] += __shfl_xor_sync(0xffffffffu, Sb[mm], o);
                Sq[mm] += __shfl_xor_sync(0xffffffffu, Sq[mm], o);
            }
            const int m = m0 + mm;
            if (lane == 0 && m < M) {
                const int acc = combine_generic<LV>(S[mm], Sb[mm], Sq[mm]);
                const size_t o = static_cast<size_t>(m) * N + n;
                if (acc_debug) acc_debug[o] = acc;
                const float y = scale_epilogue(acc, s_a[m], s_n[n]);
                if (y_bf16) static_cast<uint16_t*>(Y)[o] = f32_to_bf16_bits(y);
                else static_cast<float*>(Y)[o] = y;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// bandwidth route
// ------------------------------------------------------------------------------------------------
constexpr int kDecWarps = 8;                       // consumer warps
constexpr int kDecConsumers = kDecWarps * 32;      // 256
constexpr int kDecThreads = kDecConsumers + 32;    // + producer warp
constexpr int kQPad = 64;

template <int LV>
struct DecodeTraits {
    static constexpr int PER = codes_per_word(LV);
    static constexpr int NPL = PER / 4;                     // operand registers per packed word
    static constexpr int QBYTES = kChunkWords * PER;        // q_a bytes per token per stage
    static constexpr int QSTRIDE = QBYTES + kQPad;
    static constexpr int NQP = (LV == QIFT_LEVELS_POT) ? 2 : 1;  // q planes (POT: 5q and 6q)
    static constexpr int BPT = QBYTES / kDecConsumers;      // q bytes per consumer thread per token
};

struct DecodeParams {
    const uint32_t* packed;
    const float* s_n;
    const int8_t* q_a;
    const float* s_a;
    void* Y;
    int32_t* acc_debug;
    int M, N, K;
    int y_bf16;
    int stages;
};

__host__ __device__ inline size_t decode_stage_bytes(int lv, int rt, int M) {
    const int per = codes_per_word(lv);
    const int nqp = (lv == QIFT_LEVELS_POT) ? 2 : 1;
    return static_cast<size_t>(rt) * kTileBytes + static_cast<size_t>(nqp) * M * (kChunkWords * per + kQPad);
}
__host__ __device__ inline size_t decode_smem_bytes(int lv, int rt, int nt, int M, int stages) {
    return stages * decode_stage_bytes(lv, rt, M) + static_cast<size_t>(kDecWarps) * rt * nt * 128 * 4  // reduce
           + 2 * stages * 8 + 16 * 4 + 16;  // barriers, sum-q, flag
}

// Per-byte k*q on four packed s8 values (|k*q| < 128).
__device__ __forceinline__ uint32_t scale_s8x4(uint32_t q, int k) {
    uint32_t r = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int v = static_cast<int>(static_cast<int8_t>(q >> (8 * i))) * k;
        r |= (static_cast<uint32_t>(v) & 0xffu) << (8 * i);
    }
    return r;
}

__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers) : "memory"); }

template <int LV, int NT, int RT>
__global__ void __launch_bounds__(kDecThreads)
linear_decode_kernel(const DecodeParams p) {
    using T = DecodeTraits<LV>;
    constexpr int ROWS = 16 * RT;
    extern __shared__ __align__(128) unsigned char smem[];
    const int M = p.M;
    const size_t stage_bytes = decode_stage_bytes(LV, RT, M);
    const int stages = p.stages;
    unsigned char* ring = smem;
    int* red = reinterpret_cast<int*>(smem + stages * stage_bytes);                 // [warp][RT*NT][16][8]
    uint64_t* full = reinterpret_cast<uint64_t*>(red + kDecWarps * RT * NT * 128);  // [stages]
    uint64_t* empty = full + stages;                                                // [stages]
    int* sumq = reinterpret_cast<int*>(empty + stages);                             // [16]
    volatile int* fail = sumq + 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int words_per_row = p.K / T::PER;
    const int nchunks = (words_per_row + kChunkWords - 1) / kChunkWords;
    const int n0 = blockIdx.x * ROWS;
    const int rows_valid = min(ROWS, p.N - n0);

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kDecWarps);
        }
        mbar_fence_init();
    }
    if (tid < 16) sumq[tid] = 0;
    if (tid == 16) *fail = 0;
    __syncthreads();

    if (warp == kDecWarps) {
        // ---------------------------------------------------------------- producer warp
        const int pitch = round_up16(words_per_row);
        const unsigned char* wbase = reinterpret_cast<const unsigned char*>(p.packed) +
                                     static_cast<size_t>(n0) * pitch * 4;  // first tile of the first row block
        const size_t rb_bytes = static_cast<size_t>(16) * pitch * 4;
        const int tiles_valid = (rows_valid + 15) / 16;
        auto chunk_words = [&](int c) { return min(kChunkWords, words_per_row - c * kChunkWords); };
        auto issue_w = [&](int c, int s) {  // one bulk copy per 16-row tile
            const uint32_t bytes = chunk_words(c) * 16 * 4;
            unsigned char* dst = ring + s * stage_bytes;
            if (lane < tiles_valid)
                bulk_g2s(dst + lane * kTileBytes, wbase + lane * rb_bytes + static_cast<size_t>(c) * kTileBytes, bytes, &full[s]);
        };
        auto issue_q = [&](int c, int s) {
            const uint32_t seg = chunk_words(c) * T::PER;
            unsigned char* dst = ring + s * stage_bytes + RT * kTileBytes;
            for (int m = lane; m < M; m += 32)
                bulk_g2s(dst + m * T::QSTRIDE, p.q_a + static_cast<size_t>(m) * p.K + static_cast<size_t>(c) * T::QBYTES, seg,
                         &full[s]);
        };
        auto expect = [&](int c, int s) {
            if (lane == 0) mbar_expect_tx(&full[s], chunk_words(c) * (64 * tiles_valid + T::PER * M));
            __syncwarp();
        };
        const int npre = min(stages, nchunks);
        for (int c = 0; c < npre; ++c) {
            expect(c, c);
            issue_w(c, c);  // weights do not depend on the previous kernel
        }
        pdl_wait();
        for (int c = 0; c < npre; ++c) issue_q(c, c);
        for (int c = npre; c < nchunks; ++c) {
            const int s = c % stages;
            if (!mbar_wait(&empty[s], ((c / stages) - 1) & 1, 1)) break;
            expect(c, s);
            issue_w(c, s);
            issue_q(c, s);
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    pdl_wait();
    const int g = lane >> 2, cq = lane & 3;
    int acc[RT][NT][T::NPL][4];
#pragma unroll
    for (int a = 0; a < RT; ++a)
#pragma unroll
        for (int b = 0; b < NT; ++b)
#pragma unroll
            for (int t = 0; t < T::NPL; ++t)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[a][b][t][i] = 0;
    int sq[8 * NT];
#pragma unroll
    for (int i = 0; i < 8 * NT; ++i) sq[i] = 0;
    bool ok = true;

    for (int c = 0; c < nchunks; ++c) {
        const int s = c % stages;
        if (!mbar_wait(&full[s], (c / stages) & 1, 2)) {
            ok = false;
            break;
        }
        const int cw = min(kChunkWords, words_per_row - c * kChunkWords);
        unsigned char* wst = ring + s * stage_bytes;
        unsigned char* qst = wst + RT * kTileBytes;

        // sum of q per token (and the 5q / 6q planes of POT): every consumer thread owns BPT bytes
        {
            const int off = tid * T::BPT;
            if (off < cw * T::PER) {
#pragma unroll
                for (int m = 0; m < 8 * NT; ++m) {
                    if (m < M) {
                        uint32_t* qp = reinterpret_cast<uint32_t*>(qst + m * T::QSTRIDE + off);
#pragma unroll
                        for (int i = 0; i < T::BPT / 4; ++i) {
                            const uint32_t v = qp[i];
                            sq[m] = dp4a_us(0x01010101u, v, sq[m]);
                            if constexpr (LV == QIFT_LEVELS_POT) {
                                qp[i] = scale_s8x4(v, 5);
                                reinterpret_cast<uint32_t*>(qst + (M + m) * T::QSTRIDE + off)[i] = scale_s8x4(v, 6);
                            }
                        }
                    }
                }
            }
            if constexpr (LV == QIFT_LEVELS_POT) consumer_bar_sync();
        }

        if (16 * warp < cw) {
            // B operands: the lane's four words cover 4*PER consecutive q bytes of token g (+8)
            uint32_t qb[NT][T::NQP][4 * T::NPL];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int m = nt * 8 + g;
#pragma unroll
                for (int pl = 0; pl < T::NQP; ++pl) {
                    if (m < M) {
                        const uint4* src = reinterpret_cast<const uint4*>(qst + (pl * M + m) * T::QSTRIDE +
                                                                          (16 * warp + 4 * cq) * T::PER);
#pragma unroll
                        for (int i = 0; i < T::NPL; ++i) {
                            const uint4 v = src[i];
                            qb[nt][pl][4 * i] = v.x, qb[nt][pl][4 * i + 1] = v.y;
                            qb[nt][pl][4 * i + 2] = v.z, qb[nt][pl][4 * i + 3] = v.w;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 4 * T::NPL; ++i) qb[nt][pl][i] = 0;
                    }
                }
            }
#pragma unroll
            for (int rt = 0; rt < RT; ++rt) {
                // tile order: group ((slice*2 + half)*32 + lane); slice = this warp, half = rows g / g+8
                const uint4 wa = *reinterpret_cast<const uint4*>(wst + rt * kTileBytes + ((2 * warp) * 32 + lane) * 16);
                const uint4 wb = *reinterpret_cast<const uint4*>(wst + rt * kTileBytes + ((2 * warp + 1) * 32 + lane) * 16);
                const uint32_t a_lo[4] = {wa.x, wa.y, wa.z, wa.w};
                const uint32_t a_hi[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                for (int pr = 0; pr < 2; ++pr) {
                    const int i0 = 2 * pr, i1 = 2 * pr + 1;
#pragma unroll
                    for (int t = 0; t < T::NPL; ++t) {
                        if constexpr (LV == QIFT_LEVELS_INT4) {
                            const uint32_t msk = 0x0f0f0f0fu << (4 * t), flip = 0x08080808u << (4 * t);
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt)
                                mma_u8s8(acc[rt][nt][t], (a_lo[i0] & msk) ^ flip, (a_hi[i0] & msk) ^ flip,
                                         (a_lo[i1] & msk) ^ flip, (a_hi[i1] & msk) ^ flip,
                                         qb[nt][0][i0 * T::NPL + t], qb[nt][0][i1 * T::NPL + t]);
                        } else if constexpr (LV == QIFT_LEVELS_POT) {
                            // 10*b1 + 6*b0 = 2*(level + 4): bit 1 against the 5q plane, bit 0 against 6q
                            const uint32_t m1 = 0x02020202u << (2 * t), m0 = 0x01010101u << (2 * t);
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                mma_u8s8(acc[rt][nt][t], a_lo[i0] & m1, a_hi[i0] & m1, a_lo[i1] & m1, a_hi[i1] & m1,
                                         qb[nt][0][i0 * T::NPL + t], qb[nt][0][i1 * T::NPL + t]);
                                mma_u8s8(acc[rt][nt][t], a_lo[i0] & m0, a_hi[i0] & m0, a_lo[i1] & m0, a_hi[i1] & m0,
                                         qb[nt][1][i0 * T::NPL + t], qb[nt][1][i1 * T::NPL + t]);
                            }
                        } else {
                            const uint32_t msk = 0x03030303u << (2 * t);
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt)
                                mma_u8s8(acc[rt][nt][t], a_lo[i0] & msk, a_hi[i0] & msk, a_lo[i1] & msk, a_hi[i1] & msk,
                                         qb[nt][0][i0 * T::NPL + t], qb[nt][0][i1 * T::NPL + t]);
                        }
                    }
                }
            }
        }
        if (nchunks > stages) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
    }
    if (!ok) *fail = 1;

    // per-warp partials: divide the t-planes out (exact) and park them for the cross-warp sum
    constexpr int SH = (LV == QIFT_LEVELS_INT4) ? 4 : 2;
#pragma unroll
    for (int rt = 0; rt < RT; ++rt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            int* dst = red + ((warp * RT + rt) * NT + nt) * 128;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int v = 0;
#pragma unroll
                for (int t = 0; t < T::NPL; ++t) v += acc[rt][nt][t][i] >> (SH * t);
                const int row = g + ((i & 2) ? 8 : 0), tok = 2 * cq + (i & 1);
                dst[row * 8 + tok] = v;
            }
        }
#pragma unroll
    for (int m = 0; m < 8 * NT; ++m) {
        if (m < M) {
            int v = sq[m];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) atomicAdd(&sumq[m], v);
        }
    }
    consumer_bar_sync();
    if (*fail) return;

    for (int o = tid; o < ROWS * M; o += kDecConsumers) {
        const int row = o % ROWS, m = o / ROWS;
        const int n = n0 + row;
        if (n >= p.N) continue;
        const int rt = row / 16, r = row % 16, nt = m / 8, tk = m % 8;
        int S = 0;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) S += red[((w * RT + rt) * NT + nt) * 128 + r * 8 + tk];
        const int Sq = sumq[m];
        int acc_v;
        if constexpr (LV == QIFT_LEVELS_MNZ) acc_v = 2 * S - 3 * Sq;
        else if constexpr (LV == QIFT_LEVELS_SYM) acc_v = S - 2 * Sq;
        else if constexpr (LV == QIFT_LEVELS_POT) acc_v = (S >> 1) - 4 * Sq;
        else acc_v = S - 8 * Sq;
        const size_t idx = static_cast<size_t>(m) * p.N + n;
        if (p.acc_debug) p.acc_debug[idx] = acc_v;
        const float y = scale_epilogue(acc_v, p.s_a[m], p.s_n[n]);
        if (p.y_bf16) static_cast<uint16_t*>(p.Y)[idx] = f32_to_bf16_bits(y);
        else static_cast<float*>(p.Y)[idx] = y;
    }
}

}  // namespace qift

// Decode-path product kernels (M <= 16): stream the packed codes from HBM once, decode in
// registers, accumulate exactly in INT32, apply the scales in the epilogue.
//
//  * linear_generic_kernel: one warp per output channel, dp4a.  Any M, any K; the slow, simple route.
//  * linear_decode_kernel:  the bandwidth route.  A producer warp stages 16-row x 128-word tiles of
//    packed weights (8 KB each, contiguous in memory: one cp.async.bulk per tile), and the matching
//    slice of q_a, into a shared-memory ring guarded by mbarriers.  The weight copies are issued BEFORE the programmatic-dependent-launch
//    wait, so in a stream of such launches the next layer's weights are in flight while the previous
//    layer finishes.  Eight consumer warps split each slab along K; a lane turns a packed word into
//    u8 operand registers with one logic op each (w & (0x03030303 << 2t) = code * 4^t, which the
//    integer tensor-core instruction mma.sync.m16n8k32.u8.s8 multiplies against q_a directly) and keeps
//    one accumulator set per place value; the exact division by the place value, the affine level map
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
    if constexpr (LV == QIFT_LEVELS_INT3) return S - 4 * Sb1;          // S over the two low bits, Sb1 over the third
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
            uint32_t w, wh = 0;
            if constexpr (LV == QIFT_LEVELS_INT3) {
                w = packed[int3_low_address(n, j, pitch)];
                wh = packed[int3_high_address(n, j, pitch)];
            } else {
                w = packed[packed_word_address(n, j, pitch)];
            }
#pragma unroll
            for (int t = 0; t < NPL; ++t) {
                uint32_t a, hb = 0;
                if constexpr (LV == QIFT_LEVELS_INT4) {
                    a = ((w >> (BITS * t)) & 0x0f0f0f0fu) ^ 0x08080808u;
                } else if constexpr (LV == QIFT_LEVELS_INT3) {
                    a = (w >> (BITS * t)) & 0x03030303u;
                    hb = (wh >> int3_high_shift(j, t)) & 0x01010101u;
                } else {
                    a = (w >> (BITS * t)) & 0x03030303u;
                    hb = (a >> 1) & 0x01010101u;
                }
#pragma unroll
                for (int mm = 0; mm < kGenericTokens; ++mm) {
                    if (m0 + mm < M) {
                        const uint32_t qv = q32[(m0 + mm) * qpitch + static_cast<size_t>(j) * NPL + t];
                        S[mm] = dp4a_us(a, qv, S[mm]);
                        if constexpr (LV == QIFT_LEVELS_POT || LV == QIFT_LEVELS_INT3) Sb[mm] = dp4a_us(hb, qv, Sb[mm]);
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

// How one packed word becomes tensor-core operands.  An m16n8k32 instruction has two k-halves of
// 16; a lane supplies 4 bytes of each.  Both halves are fed from the SAME word: half 0 takes code
// plane tt (w & mask), half 1 takes plane tt+1, so that the matching activations are two adjacent
// 32-bit words of q_a -- an aligned register pair, no register shuffling.  The two planes differ by
// a factor 4 (INT4: 16) in place value; either the odd plane is shifted down first (plain q_a), or
// q_a arrives with its even-plane bytes already multiplied by that factor (PRESCALED, the grouped
// path), in which case a single logic op per operand register remains.
//   accumulator sets: MNZ/SYM 2 (planes 0-1, 2-3), POT 4 (two code bits x two plane pairs), INT4 1
template <int LV>
struct DecodeTraits {
    static constexpr int PER = codes_per_word(LV);
    static constexpr int NPL = PER / 4;                     // 32-bit q words per packed word
    static constexpr int QBYTES = kChunkWords * PER;        // q_a bytes per token per stage
    static constexpr int QSTRIDE = QBYTES + kQPad;
    static constexpr int BPT = QBYTES / kDecConsumers;      // q bytes per consumer thread per token
    static constexpr int NACC = (LV == QIFT_LEVELS_INT4) ? 1 : (LV == QIFT_LEVELS_POT) ? 4 : (LV == QIFT_LEVELS_INT3) ? 6 : 2;
};

// Place value of accumulator set `a` (a power of two; the set holds scale * sum code*q exactly).
template <int LV, bool PRESCALED>
__host__ __device__ constexpr int acc_shift(int a) {
    if (LV == QIFT_LEVELS_INT4) return PRESCALED ? 4 : 0;
    if (LV == QIFT_LEVELS_POT) {  // sets: 0,1 = code bit 1 (planes 0-1, 2-3); 2,3 = code bit 0
        const int bit1 = (a < 2) ? 1 : 0;
        return bit1 + 4 * (a & 1) + (PRESCALED ? 2 : 0);
    }
    if (LV == QIFT_LEVELS_INT3 && a >= 2) {  // sets 2..5: the high plane (prescaled activations only), bit pairs (0,2) (1,3) (4,6) (5,7)
        return 2 + (a - 2) + ((a >= 4) ? 2 : 0);
    }
    return 4 * a + (PRESCALED ? 2 : 0);
}

// Exact level sum from the accumulator sets and sum_k q:  acc = sum_k level(code_k) * q_k.
template <int LV, bool PRESCALED, int NACC>
__device__ __forceinline__ int level_sum(const int (&v)[NACC], int Sq) {
    if constexpr (LV == QIFT_LEVELS_INT4) {
        return (v[0] >> acc_shift<LV, PRESCALED>(0)) - 8 * Sq;  // code' = nibble ^ 8 = level + 8
    } else if constexpr (LV == QIFT_LEVELS_INT3) {               // level = (c & 3) - 4 (c >> 2)
        const int lo = (v[0] >> acc_shift<LV, PRESCALED>(0)) + (v[1] >> acc_shift<LV, PRESCALED>(1));
        const int hi = (v[2] >> acc_shift<LV, PRESCALED>(2)) + (v[3] >> acc_shift<LV, PRESCALED>(3)) +
                       (v[4] >> acc_shift<LV, PRESCALED>(4)) + (v[5] >> acc_shift<LV, PRESCALED>(5));
        return lo - 4 * hi;
    } else if constexpr (LV == QIFT_LEVELS_POT) {                // level = 5*b1 + 3*b0 - 4
        const int b1 = (v[0] >> acc_shift<LV, PRESCALED>(0)) + (v[1] >> acc_shift<LV, PRESCALED>(1));
        const int b0 = (v[2] >> acc_shift<LV, PRESCALED>(2)) + (v[3] >> acc_shift<LV, PRESCALED>(3));
        return 5 * b1 + 3 * b0 - 4 * Sq;
    } else {
        const int S = (v[0] >> acc_shift<LV, PRESCALED>(0)) + (v[1] >> acc_shift<LV, PRESCALED>(1));
        return (LV == QIFT_LEVELS_MNZ) ? 2 * S - 3 * Sq : S - 2 * Sq;  // level = 2c - 3  /  c - 2
    }
}

// One mma step of a warp: its four words of rows g (wa) and g+8 (wb) against the q words in qb
// (qb[NPL*i + t] = q word of plane t of word i).
template <int LV, int NT, bool PRESCALED>
__device__ __forceinline__ void mma_tile_step(int (&acc)[NT][DecodeTraits<LV>::NACC][4], const uint4 wa, const uint4 wb,
                                              const uint32_t (&qb)[NT][4 * DecodeTraits<LV>::NPL]) {
    constexpr int NPL = DecodeTraits<LV>::NPL;
    const uint32_t lo[4] = {wa.x, wa.y, wa.z, wa.w};
    const uint32_t hi[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if constexpr (LV == QIFT_LEVELS_INT4) {
            const uint32_t lo1 = PRESCALED ? lo[i] : (lo[i] >> 4), hi1 = PRESCALED ? hi[i] : (hi[i] >> 4);
            constexpr uint32_t m1 = PRESCALED ? 0xf0f0f0f0u : 0x0f0f0f0fu, f1 = PRESCALED ? 0x80808080u : 0x08080808u;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                mma_u8s8(acc[nt][0], (lo[i] & 0x0f0f0f0fu) ^ 0x08080808u, (hi[i] & 0x0f0f0f0fu) ^ 0x08080808u, (lo1 & m1) ^ f1,
                         (hi1 & m1) ^ f1, qb[nt][NPL * i], qb[nt][NPL * i + 1]);
        } else {
            const uint32_t lo2 = lo[i] >> 2, hi2 = hi[i] >> 2;  // unused when PRESCALED
#pragma unroll
            for (int tt = 0; tt < 4; tt += 2) {
                if constexpr (LV == QIFT_LEVELS_POT) {
#pragma unroll
                    for (int bit = 1; bit >= 0; --bit) {
                        const uint32_t m0 = (bit ? 0x02020202u : 0x01010101u) << (2 * tt);
                        const uint32_t m1 = PRESCALED ? (m0 << 2) : m0;
                        const uint32_t l1 = PRESCALED ? lo[i] : lo2, h1 = PRESCALED ? hi[i] : hi2;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            mma_u8s8(acc[nt][(bit ? 0 : 2) + tt / 2], lo[i] & m0, hi[i] & m0, l1 & m1, h1 & m1, qb[nt][NPL * i + tt],
                                     qb[nt][NPL * i + tt + 1]);
                    }
                } else {
                    const uint32_t m0 = 0x03030303u << (2 * tt);
                    const uint32_t m1 = PRESCALED ? (m0 << 2) : m0;
                    const uint32_t l1 = PRESCALED ? lo[i] : lo2, h1 = PRESCALED ? hi[i] : hi2;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        mma_u8s8(acc[nt][tt / 2], lo[i] & m0, hi[i] & m0, l1 & m1, h1 & m1, qb[nt][NPL * i + tt],
                                 qb[nt][NPL * i + tt + 1]);
                }
            }
        }
    }
}

// Three-bit codes: the low plane is a two-bit word like any other (sets 0, 1); the high plane adds, per low word, two
// products whose operands are single bits of the high word.  Its bit order puts planes t and t+1 (t even) of a low
// word two positions apart, so with the even planes' activations prescaled by four both halves of an instruction
// carry the place value 4 * 2^u: u = 0, 1 for the even low word of a pair (sets 2, 3), 4, 5 for the odd one (sets 4, 5).
// wh = {high words 0, 1 of row g, high words 0, 1 of row g+8} of the lane's four low words.
template <int NT>
__device__ __forceinline__ void mma_tile_step_int3(int (&acc)[NT][6][4], const uint4 wa, const uint4 wb, const uint4 wh,
                                                   const uint32_t (&qb)[NT][16]) {
    const uint32_t lo[4] = {wa.x, wa.y, wa.z, wa.w};
    const uint32_t hi[4] = {wb.x, wb.y, wb.z, wb.w};
    const uint32_t hl[2] = {wh.x, wh.y}, hh[2] = {wh.z, wh.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int tt = 0; tt < 4; tt += 2) {
            const uint32_t m0 = 0x03030303u << (2 * tt), m1 = m0 << 2;
            const uint32_t b0 = 0x01010101u << (4 * (i & 1) + tt / 2), b1 = b0 << 2;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                mma_u8s8(acc[nt][tt / 2], lo[i] & m0, hi[i] & m0, lo[i] & m1, hi[i] & m1, qb[nt][4 * i + tt], qb[nt][4 * i + tt + 1]);
                mma_u8s8(acc[nt][2 + 2 * (i & 1) + tt / 2], hl[i >> 1] & b0, hh[i >> 1] & b0, hl[i >> 1] & b1, hh[i >> 1] & b1,
                         qb[nt][4 * i + tt], qb[nt][4 * i + tt + 1]);
            }
        }
    }
}

// PoT levels {-4,-1,+1,+4} are not affine in the code, so the masked-code operand above needs one product per code
// BIT.  Where the activation bytes can be laid out to order (the grouped row-split kernel), the levels themselves
// become the operand instead: a byte-permute instruction is a four-entry table lookup on four selector nibbles,
// and (w >> s) & 0x3333 holds four codes of a packed word as nibbles.  One word yields four signed-byte operand
// registers whose bytes are the levels of codes k = {0,8,1,9}, {4,12,5,13}, {2,10,3,11}, {6,14,7,15} of the word;
// the quantizer writes each 16-byte activation group in the same order (pot_lut_order), unscaled.  One product
// instruction per 512 codes and token tile, one accumulator set, no correction term.
__device__ __forceinline__ void pot_lut_operands(uint32_t w, uint32_t (&a)[4]) {
    constexpr uint32_t kLut = 0x0401fffcu;  // bytes: level of code 0, 1, 2, 3
    const uint32_t y = w & 0x33333333u, z = (w >> 2) & 0x33333333u;
    a[0] = __byte_perm(kLut, kLut, y);
    a[1] = __byte_perm(kLut, kLut, z);
    a[2] = __byte_perm(kLut, kLut, y >> 16);
    a[3] = __byte_perm(kLut, kLut, z >> 16);
}

// The matching order of a 16-byte activation group (four words of four consecutive-k bytes each).
__device__ __forceinline__ uint4 pot_lut_order(uint4 q) {
    return make_uint4(__byte_perm(q.x, q.z, 0x5140), __byte_perm(q.y, q.w, 0x5140), __byte_perm(q.x, q.z, 0x7362),
                      __byte_perm(q.y, q.w, 0x7362));
}

template <int NT>
__device__ __forceinline__ void mma_tile_step_pot_lut(int (&acc)[NT][1][4], const uint4 wa, const uint4 wb,
                                                      const uint32_t (&qb)[NT][16]) {
    const uint32_t lo[4] = {wa.x, wa.y, wa.z, wa.w};
    const uint32_t hi[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t al[4], ah[4];
        pot_lut_operands(lo[i], al);
        pot_lut_operands(hi[i], ah);
#pragma unroll
        for (int p = 0; p < 2; ++p)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                mma_s8s8(acc[nt][0], al[2 * p], ah[2 * p], al[2 * p + 1], ah[2 * p + 1], qb[nt][4 * i + 2 * p], qb[nt][4 * i + 2 * p + 1]);
    }
}

// One packed word of rows g (lo) and g+8 (hi) against the NPL activation words that belong to it, grouped-path
// layouts (prescaled even planes, or PoT table order with POT_LUT).  The operand logic does not depend on the token
// tile: called in a loop over token tiles it is computed once.
template <int LV, bool POT_LUT, int NACC>
__device__ __forceinline__ void mma_word(int (&acc)[NACC][4], uint32_t lo, uint32_t hi, const uint32_t (&q)[DecodeTraits<LV>::NPL]) {
    if constexpr (LV == QIFT_LEVELS_INT4) {
        mma_u8s8(acc[0], (lo & 0x0f0f0f0fu) ^ 0x08080808u, (hi & 0x0f0f0f0fu) ^ 0x08080808u, (lo & 0xf0f0f0f0u) ^ 0x80808080u,
                 (hi & 0xf0f0f0f0u) ^ 0x80808080u, q[0], q[1]);
    } else if constexpr (POT_LUT) {
        uint32_t al[4], ah[4];
        pot_lut_operands(lo, al);
        pot_lut_operands(hi, ah);
        mma_s8s8(acc[0], al[0], ah[0], al[1], ah[1], q[0], q[1]);
        mma_s8s8(acc[0], al[2], ah[2], al[3], ah[3], q[2], q[3]);
    } else if constexpr (LV == QIFT_LEVELS_POT) {
#pragma unroll
        for (int tt = 0; tt < 4; tt += 2)
#pragma unroll
            for (int bit = 1; bit >= 0; --bit) {
                const uint32_t m0 = (bit ? 0x02020202u : 0x01010101u) << (2 * tt), m1 = m0 << 2;
                mma_u8s8(acc[(bit ? 0 : 2) + tt / 2], lo & m0, hi & m0, lo & m1, hi & m1, q[tt], q[tt + 1]);
            }
    } else {
#pragma unroll
        for (int tt = 0; tt < 4; tt += 2) {
            const uint32_t m0 = 0x03030303u << (2 * tt), m1 = m0 << 2;
            mma_u8s8(acc[tt / 2], lo & m0, hi & m0, lo & m1, hi & m1, q[tt], q[tt + 1]);
        }
    }
}

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
    return static_cast<size_t>(rt) * kTileBytes + static_cast<size_t>(M) * (kChunkWords * codes_per_word(lv) + kQPad);
}
__host__ __device__ inline size_t decode_smem_bytes(int lv, int rt, int nt, int M, int stages) {
    const int nacc = (lv == QIFT_LEVELS_INT4) ? 1 : (lv == QIFT_LEVELS_POT) ? 4 : (lv == QIFT_LEVELS_INT3) ? 6 : 2;
    return stages * decode_stage_bytes(lv, rt, M) + static_cast<size_t>(kDecWarps) * rt * nt * nacc * 128 * 4  // reduce
           + 2 * stages * 8 + 16 * 4 + 16;  // barriers, sum-q, flag
}

__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kDecConsumers) : "memory"); }

template <int LV, int NT, int RT>
__global__ void __launch_bounds__(kDecThreads)
linear_decode_kernel(const DecodeParams p) {
    using T = DecodeTraits<LV>;
    constexpr int ROWS = 16 * RT;
    constexpr int FR = RT * NT * T::NACC;  // accumulator fragments per warp
    extern __shared__ __align__(128) unsigned char smem[];
    const int M = p.M;
    const size_t stage_bytes = decode_stage_bytes(LV, RT, M);
    const int stages = p.stages;
    unsigned char* ring = smem;
    int* red = reinterpret_cast<int*>(smem + stages * stage_bytes);   // [warp][RT][NT][NACC][16][8]
    uint64_t* full = reinterpret_cast<uint64_t*>(red + kDecWarps * FR * 128);  // [stages]
    uint64_t* empty = full + stages;                                           // [stages]
    int* sumq = reinterpret_cast<int*>(empty + stages);                        // [16]
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
    int acc[RT][NT][T::NACC][4];
#pragma unroll
    for (int a = 0; a < RT; ++a)
#pragma unroll
        for (int b = 0; b < NT; ++b)
#pragma unroll
            for (int t = 0; t < T::NACC; ++t)
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

        // sum of q per token: every consumer thread owns BPT bytes of each token's slice
        {
            const int off = tid * T::BPT;
            if (off < cw * T::PER) {
#pragma unroll
                for (int m = 0; m < 8 * NT; ++m) {
                    if (m < M) {
                        const uint32_t* qp = reinterpret_cast<const uint32_t*>(qst + m * T::QSTRIDE + off);
#pragma unroll
                        for (int i = 0; i < T::BPT / 4; ++i) sq[m] = dp4a_us(0x01010101u, qp[i], sq[m]);
                    }
                }
            }
        }

        if (16 * warp < cw) {
            // B operands: the lane's four words cover 4*PER consecutive q bytes of token g (+8)
            uint32_t qb[NT][4 * T::NPL];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int m = nt * 8 + g;
                if (m < M) {
                    const uint4* src = reinterpret_cast<const uint4*>(qst + m * T::QSTRIDE + (16 * warp + 4 * cq) * T::PER);
#pragma unroll
                    for (int i = 0; i < T::NPL; ++i) {
                        const uint4 v = src[i];
                        qb[nt][4 * i] = v.x, qb[nt][4 * i + 1] = v.y, qb[nt][4 * i + 2] = v.z, qb[nt][4 * i + 3] = v.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 4 * T::NPL; ++i) qb[nt][i] = 0;
                }
            }
#pragma unroll
            for (int rt = 0; rt < RT; ++rt) {
                // tile order: group ((slice*2 + half)*32 + lane); slice = this warp, half = rows g / g+8
                const uint4 wa = *reinterpret_cast<const uint4*>(wst + rt * kTileBytes + ((2 * warp) * 32 + lane) * 16);
                const uint4 wb = *reinterpret_cast<const uint4*>(wst + rt * kTileBytes + ((2 * warp + 1) * 32 + lane) * 16);
                mma_tile_step<LV, NT, false>(acc[rt], wa, wb, qb);
            }
        }
        if (nchunks > stages) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
    }
    if (!ok) *fail = 1;

    // per-warp partials, parked for the cross-warp sum
#pragma unroll
    for (int rt = 0; rt < RT; ++rt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int a = 0; a < T::NACC; ++a) {
                int* dst = red + (((warp * RT + rt) * NT + nt) * T::NACC + a) * 128;
#pragma unroll
                for (int i = 0; i < 4; ++i) dst[(g + ((i & 2) ? 8 : 0)) * 8 + 2 * cq + (i & 1)] = acc[rt][nt][a][i];
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
        int v[T::NACC];
#pragma unroll
        for (int a = 0; a < T::NACC; ++a) {
            int S = 0;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) S += red[(((w * RT + rt) * NT + nt) * T::NACC + a) * 128 + r * 8 + tk];
            v[a] = S;
        }
        const int acc_v = level_sum<LV, false, T::NACC>(v, sumq[m]);
        const size_t idx = static_cast<size_t>(m) * p.N + n;
        if (p.acc_debug) p.acc_debug[idx] = acc_v;
        const float y = scale_epilogue(acc_v, p.s_a[m], p.s_n[n]);
        if (p.y_bf16) static_cast<uint16_t*>(p.Y)[idx] = f32_to_bf16_bits(y);
        else static_cast<float*>(p.Y)[idx] = y;
    }
}

}  // namespace qift

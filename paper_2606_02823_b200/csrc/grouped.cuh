// Grouped decode path: ONE persistent launch serves a whole list of independent layer problems
// (all of one level set and one token count M <= 64), e.g. every linear module of a decode step.
//
// A single W2 matrix is 1-15 MB, i.e. 0.15-2 us of HBM time: no per-matrix launch can reach a
// bandwidth steady state.  Here the work list (problem, 16*RT-row block) is dealt round-robin to a
// grid of resident CTAs; in each CTA a producer warp streams 8 KB tiles of packed codes (one
// cp.async.bulk each, plus the matching q_a slices) through a ring of shared-memory stages guarded
// by mbarriers and keeps running ahead across item boundaries, so HBM requests never drain between
// matrices; eight consumer warps do the same in-register decode + mma.sync as the per-call kernel.
#pragma once

#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "decode.cuh"
#include "rotate_quant.cuh"

namespace qift {

struct GroupHeader {
    uint32_t magic;
    int count;          // problems
    int M;              // token rows of every problem
    int levels;
    int y_bf16;
    int x_bf16;
    float clip;
    int total_items;    // row blocks over all problems
    int rows_per_item;  // 16 * RT
    int max_k;
    int any_kron;       // some problem's had_block selects the full-dimension rotation (K = 28 * 2^p)
    int q_chunk_bytes;  // 0: q_a row-major [M][K]; else chunk-major for the row-split kernel (ChunkMajorDst)
    int q_pot_lut;      // q_a unscaled, bytes of each 16-byte group in pot_lut_order (PoT on the row-split kernel)
    int reserved[3];
};
static_assert(sizeof(GroupHeader) == 64, "header is one 64-byte record");

struct GroupProblemDev {
    const void* X;          // [M,K] activations (fp32 or bf16), input of the quantizer
    const uint32_t* packed;
    const float* s_n;
    int8_t* q_a;            // [M,K] written by the grouped quantizer, read by the product
    float* s_a;             // [M]
    void* Y;                // [M,N]
    int32_t* acc_debug;     // [M,N] or null
    int N, K, had_block;
    int item_begin;         // first work item of this problem
    float inv_sqrt_b;
    int quant_src;          // problem whose quantized activation (q_a, s_a, sum of q) this one uses: itself, or an earlier one
                            // with the same X, q_a, s_a, K and rotation (q/k/v, gate/up: one quantization for all)
    int pad[4];
};
static_assert(sizeof(GroupProblemDev) == 96, "problem record is 96 bytes");

constexpr int kGroupMaxM = 128;    // token rows of a plan (65 .. 128: the tcgen05 kernel only); also the row length of the token-sum table
constexpr int kWideMaxM = 64;      // token rows the mma.sync row-split kernel takes (eight token tiles)
constexpr uint32_t kGroupMagic = 0x51494654u;

// ------------------------------------------------------------------------------------------------
// grouped quantizer: one CTA per (problem, token row); also leaves sum_k q_a for the product kernel
// ------------------------------------------------------------------------------------------------
// q_a is written PRESCALED for the product kernel (see mma_tile_step): with two-bit weights the
// bytes of the even code planes (k % 16 in 0..3 or 8..11) hold 4*q, with INT4 weights the bytes of
// plane 0 (k % 8 in 0..3) hold 16*q; sumq holds the plain sum of q.
// Layout of q_a for the row-split product kernel, which stages one K-chunk of ALL tokens per pipeline stage: chunk
// after chunk, inside a chunk token after token (so a stage is one contiguous piece of memory, one bulk copy).
// Inside a token's chunk the 16-byte groups are permuted so that the product kernel's reads are free of bank
// conflicts although every lane visits its groups in the same order: a quarter-warp of that kernel reads, in one
// instruction, group index i of the 64-byte blocks cq = 0..3 of tokens g and g+1.  Blocks two apart would share
// their banks, as would the two tokens; so the group index is XORed with 2 in every other PAIR of blocks (two-bit
// weights: four groups per block) and with 1 for odd tokens.  INT4 weights have two groups per 32-byte block and
// only the token swap.
//   byte address of group q of token m:  c = 16 q / CB,  c CB M + m min(CB, K - c CB) + 16 swizzled(q mod CB/16)
__host__ __device__ __forceinline__ int swizzled_group(int piece, int m, int two_bit) {
    const int block_pair = two_bit ? ((piece >> 3) & 1) << 1 : 0;   // bit 1 of the 64-byte block index -> bit 1 of the group index
    return piece ^ block_pair ^ (m & 1);
}
struct RowMajorPotDst {   // row-major, bytes of each 16-byte group in pot_lut_order (PoT on the tcgen05 kernel)
    int8_t* q_row;
    __device__ __forceinline__ void store(int q, uint4 v) const { reinterpret_cast<uint4*>(q_row)[q] = pot_lut_order(v); }
};
struct ChunkMajorDst {
    int8_t* q_a;
    int m, M, K, cb, pot_lut, two_bit;
    __device__ __forceinline__ void store(int q, uint4 v) const {
        if (pot_lut) v = pot_lut_order(v);
        const int c = (16 * q) / cb, piece = q - c * (cb / 16);
        const int bytes = min(cb, K - c * cb);
        *reinterpret_cast<uint4*>(q_a + static_cast<size_t>(c) * cb * M + static_cast<size_t>(m) * bytes +
                                  16 * swizzled_group(piece, m, two_bit)) = v;
    }
};

template <bool BF16_IN, bool KRON = false>
__global__ void __launch_bounds__(kRowThreads)
quantize_act_grouped_kernel(const GroupProblemDev* __restrict__ problems, int* __restrict__ sumq, int M, float clip,
                            int int4_weights, int q_chunk_bytes, int q_pot_lut, int use_single, const GroupProblemDev single) {
    extern __shared__ __align__(16) float row[];
    __shared__ float red[kRowThreads / 32 + 2];
    __shared__ int redi[kRowThreads / 32];
    pdl_launch_dependents();
    pdl_wait();
    const int p = blockIdx.x / M;
    const GroupProblemDev P = use_single ? single : problems[p];   // a per-call forward passes its one problem by value
    if (P.quant_src != p) return;  // an earlier problem quantizes this activation
    const size_t m = blockIdx.x % M;
    const int K = P.K, B = P.had_block;
    const RowScale sc = block_row_scale(load_and_transform<BF16_IN, KRON>(P.X, m, K, B, row), clip, red);
    if (threadIdx.x == 0) P.s_a[m] = (B > 1) ? __fmul_rn(sc.s_u, P.inv_sqrt_b) : sc.s_u;
    // 32-bit word i of a 16-byte group = code plane (two-bit: i; INT4: i & 1); even planes are prescaled
    const float mult = q_pot_lut ? 1.0f : int4_weights ? 16.0f : 4.0f;
    int total = q_chunk_bytes ? quantize_row<true>(row, K, sc, ChunkMajorDst{P.q_a, static_cast<int>(m), M, K, q_chunk_bytes, q_pot_lut, int4_weights ? 0 : 1}, mult, 1.0f)
                : q_pot_lut   ? quantize_row<true>(row, K, sc, RowMajorPotDst{P.q_a + m * K}, mult, 1.0f)
                              : quantize_row<true>(row, K, sc, RowMajorDst{P.q_a + m * K}, mult, 1.0f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if ((threadIdx.x & 31) == 0) redi[threadIdx.x >> 5] = total;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < kRowThreads / 32; ++w) t += redi[w];
        sumq[p * kGroupMaxM + m] = t;
    }
}

// Per-call products with 2..16 token rows take the row-split kernel as well: this kernel turns the public q_a
// ([M][K] plain bytes) into that kernel's layout in caller scratch (prescaled even planes, or PoT table order;
// chunk-major, ChunkMajorDst) and leaves the token sums.  One CTA per token row.
__global__ void __launch_bounds__(128)
relayout_act_kernel(const int8_t* __restrict__ q_a, int M, int K, int int4_weights, int q_chunk_bytes, int q_pot_lut,
                    int8_t* __restrict__ q_out, int* __restrict__ sumq) {
    __shared__ int red[4];
    pdl_launch_dependents();
    pdl_wait();
    const int m = blockIdx.x;
    const ChunkMajorDst dst{q_out, m, M, K, q_chunk_bytes, q_pot_lut, int4_weights ? 0 : 1};
    const uint4* src = reinterpret_cast<const uint4*>(q_a + static_cast<size_t>(m) * K);
    int total = 0;
    for (int q = threadIdx.x; q < K / 16; q += blockDim.x) {
        uint4 v = src[q];
        total = __dp4a(static_cast<int>(v.x), 0x01010101, __dp4a(static_cast<int>(v.y), 0x01010101, total));
        total = __dp4a(static_cast<int>(v.z), 0x01010101, __dp4a(static_cast<int>(v.w), 0x01010101, total));
        if (!q_pot_lut) {  // bytes of the even words times 4 (INT4 weights: 16); |q| <= 8, so the products fit a byte
            if (int4_weights) v.x = (v.x << 4) & 0xf0f0f0f0u, v.z = (v.z << 4) & 0xf0f0f0f0u;
            else v.x = (v.x << 2) & 0xfcfcfcfcu, v.z = (v.z << 2) & 0xfcfcfcfcu;
        }
        dst.store(q, v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = total;
    __syncthreads();
    if (threadIdx.x == 0) sumq[m] = red[0] + red[1] + red[2] + red[3];
}

// ------------------------------------------------------------------------------------------------
// grouped product
// ------------------------------------------------------------------------------------------------
struct SmemProblem {  // what the product kernel needs of a problem, 64 bytes, in shared memory
    const unsigned char* packed;
    const int8_t* q_a;
    const float* s_n;
    const float* s_a;
    void* Y;
    int32_t* acc_debug;
    int N, K;
    int item_begin;
    int index;  // row of the sum-q table: the plan position of the problem that quantized the activation
};
static_assert(sizeof(SmemProblem) == 64, "shared-memory problem record is 64 bytes");

constexpr int kGroupSlice = 256;  // problems per launch (their table lives in shared memory)

// Walks this CTA's share of the work list chunk by chunk; the producer and the consumers each run
// one and see the same sequence.  PER = codes per packed word.
// WB = bytes of one packed word column of a 16-row tile (64; 96 with the one-bit plane of the three-bit codes).
template <int PER, int CW = kChunkWords, int WB = 64>
struct GroupCursor {
    const SmemProblem* table;
    int count, item_end, rows_per_item;
    int item, p;
    const unsigned char* wbase;   // first tile of the item's first row block
    const int8_t* q_a;
    size_t rb_bytes;              // bytes between consecutive row blocks
    int N, K, n0, tiles_valid, words_per_row, nchunks;
    int chunk;

    __device__ __forceinline__ void init(const SmemProblem* t, int cnt, int item_first, int item_last, int rpi) {
        table = t, count = cnt, item_end = item_last, rows_per_item = rpi;
        item = item_first + blockIdx.x, p = 0, chunk = 0;
        load_item();
    }
    __device__ __forceinline__ bool valid() const { return item < item_end; }
    __device__ __forceinline__ void load_item() {
        if (item >= item_end) return;
        while (p + 1 < count && item >= table[p + 1].item_begin) ++p;
        const SmemProblem& P = table[p];
        N = P.N, K = P.K;
        words_per_row = K / PER;
        nchunks = (words_per_row + CW - 1) / CW;
        n0 = (item - P.item_begin) * rows_per_item;
        tiles_valid = (min(rows_per_item, N - n0) + 15) >> 4;
        const int pitch = round_up16(words_per_row);
        rb_bytes = static_cast<size_t>(pitch) * WB;
        wbase = P.packed + static_cast<size_t>(n0 >> 4) * pitch * WB;
        q_a = P.q_a;
    }
    __device__ __forceinline__ int chunk_words() const { return min(CW, words_per_row - chunk * CW); }
    __device__ __forceinline__ bool last_chunk() const { return chunk + 1 == nchunks; }
    __device__ __forceinline__ void next() {
        if (++chunk == nchunks) {
            chunk = 0;
            item += gridDim.x;
            load_item();
        }
    }
    __device__ __forceinline__ void next_item() {   // from any chunk of the item
        chunk = 0;
        item += gridDim.x;
        load_item();
    }
};

// Cross-warp reduction buffer: [warp][row tile][accumulator set][token][row], only the M live columns.
__host__ __device__ inline int grouped_red_ints(int lv, int rt, int M) {
    const int nacc = (lv == QIFT_LEVELS_INT4) ? 1 : (lv == QIFT_LEVELS_POT) ? 4 : (lv == QIFT_LEVELS_INT3) ? 6 : 2;
    return kDecWarps * rt * nacc * 16 * M;
}
__host__ __device__ inline size_t grouped_fixed_smem(int lv, int rt, int M, int count) {
    return static_cast<size_t>(count) * sizeof(SmemProblem) + 2 * static_cast<size_t>(grouped_red_ints(lv, rt, M)) * 4 + 16;
}
__host__ __device__ inline size_t grouped_smem_bytes(int lv, int rt, int M, int stages, int count) {
    return grouped_fixed_smem(lv, rt, M, count) + stages * (decode_stage_bytes(lv, rt, M) + 16);
}

struct GroupParams {
    const GroupProblemDev* problems;  // first problem of this launch's slice
    const int* sumq;                  // [plan count][kGroupMaxM]
    int first_index;                  // plan index of problems[0]
    int count;                        // problems in the slice (<= kGroupSlice)
    int item_first, item_end;         // work items of the slice
    int M, y_bf16, stages;
    int use_single;                   // the list is the one problem below (a per-call product: no plan in memory)
    GroupProblemDev single;
    const CUtensorMap* maps;          // tcgen05 kernel only: one tensor map per problem of the slice over its q_a
};

// CTAs per SM the kernel is compiled and launched for.  Nine warps per CTA and registers handed out
// to four warps at a time leave room for two CTAs only up to 96 registers per thread; the PoT
// variants (four accumulator sets) would spill at that size and run one CTA per SM instead.
template <int LV>
constexpr int grouped_ctas_per_sm() {
    return (LV == QIFT_LEVELS_POT) ? 1 : 2;
}

// M1: the single-token specialisation (only accumulator column 0 is live).
template <int LV, int NT, int RT, bool M1>
__global__ void __launch_bounds__(kDecThreads, grouped_ctas_per_sm<LV>())
linear_grouped_kernel(const GroupParams gp) {
    using T = DecodeTraits<LV>;
    constexpr int ROWS = 16 * RT;
    extern __shared__ __align__(128) unsigned char smem[];
    const int M = M1 ? 1 : gp.M;
    const int RED = grouped_red_ints(LV, RT, M);  // ints per reduction buffer
    const uint32_t stage_bytes = static_cast<uint32_t>(decode_stage_bytes(LV, RT, M));
    const int stages = gp.stages;
    unsigned char* ring = smem;
    int* red_all = reinterpret_cast<int*>(smem + stages * stage_bytes);
    SmemProblem* table = reinterpret_cast<SmemProblem*>(red_all + 2 * RED);
    uint64_t* full = reinterpret_cast<uint64_t*>(table + gp.count);
    uint64_t* empty = full + stages;
    volatile int* fail = reinterpret_cast<volatile int*>(empty + stages);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kDecWarps);
        }
        mbar_fence_init();
        *fail = 0;
    }
    // the plan was uploaded by a copy that completed before any kernel of this stream segment began
    for (int i = tid; i < gp.count; i += kDecThreads) {
        const GroupProblemDev& P = gp.problems[i];
        SmemProblem e;
        e.packed = reinterpret_cast<const unsigned char*>(P.packed);
        e.q_a = P.q_a, e.s_n = P.s_n, e.s_a = P.s_a, e.Y = P.Y, e.acc_debug = P.acc_debug;
        e.N = P.N, e.K = P.K, e.item_begin = P.item_begin, e.index = P.quant_src;
        table[i] = e;
    }
    __syncthreads();

    if (warp == kDecWarps) {
        // ---------------------------------------------------------------- producer warp
        using Cursor = GroupCursor<T::PER>;
        auto expect = [&](const Cursor& c, int s) {
            if (lane == 0) mbar_expect_tx(&full[s], c.chunk_words() * (64 * c.tiles_valid + T::PER * M));
            __syncwarp();
        };
        auto issue_w = [&](const Cursor& c, int s) {  // one bulk copy per 16-row tile
            const uint32_t bytes = c.chunk_words() * 16 * 4;
            unsigned char* dst = ring + s * stage_bytes;
            if (lane < c.tiles_valid)
                bulk_g2s(dst + lane * kTileBytes, c.wbase + lane * c.rb_bytes + static_cast<size_t>(c.chunk) * kTileBytes, bytes,
                         &full[s]);
        };
        auto issue_q = [&](const Cursor& c, int s) {
            const uint32_t seg = c.chunk_words() * T::PER;
            unsigned char* dst = ring + s * stage_bytes + RT * kTileBytes;
            for (int m = lane; m < M; m += 32)
                bulk_g2s(dst + m * T::QSTRIDE, c.q_a + static_cast<size_t>(m) * c.K + static_cast<size_t>(c.chunk) * T::QBYTES, seg,
                         &full[s]);
        };
        // the packed weights never depend on the previous kernel: fill the ring with them first
        Cursor a;
        a.init(table, gp.count, gp.item_first, gp.item_end, ROWS);
        int pre = 0;
        for (; pre < stages && a.valid(); ++pre, a.next()) {
            expect(a, pre);
            issue_w(a, pre);
        }
        pdl_wait();
        Cursor b;
        b.init(table, gp.count, gp.item_first, gp.item_end, ROWS);
        for (int i = 0; i < pre; ++i, b.next()) issue_q(b, i);
        int s = 0;
        uint32_t ph = 0;  // parity of the consumers' release this slot is waiting for
        for (; b.valid(); b.next()) {
            if (!mbar_wait(&empty[s], ph, 3)) break;
            expect(b, s);
            issue_w(b, s);
            issue_q(b, s);
            if (++s == stages) s = 0, ph ^= 1;
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    pdl_wait();
    const int g = lane >> 2, cq = lane & 3;
    GroupCursor<T::PER> cur;
    cur.init(table, gp.count, gp.item_first, gp.item_end, ROWS);
    bool ok = true;
    int s = 0;
    uint32_t ph = 0, item_no = 0;
    // epilogue role of this thread: output (row, token) = (tid % ROWS, tid / ROWS); ROWS * M <= 256
    const int e_row = tid % ROWS, e_m = tid / ROWS;
    const uint32_t a_off = (2 * warp * 32 + lane) * 16;           // this lane's group inside a tile (rows g), +512 for g+8
    const uint32_t q_off = (16 * warp + 4 * cq) * T::PER;         // this lane's q bytes inside a token's slice

    for (; cur.valid() && ok; ++item_no) {
        int* red = red_all + RED * (item_no & 1);
        int acc[RT][NT][T::NACC][4];
#pragma unroll
        for (int a = 0; a < RT; ++a)
#pragma unroll
            for (int b = 0; b < NT; ++b)
#pragma unroll
                for (int t = 0; t < T::NACC; ++t)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[a][b][t][i] = 0;
        const SmemProblem* P = &table[cur.p];
        const int n0 = cur.n0;
        const int e_n = n0 + e_row;
        const bool e_on = (e_m < M) && (e_n < cur.N);
        // fetch what the epilogue needs now; the loads complete under the chunk loop
        float e_sn = 0.0f, e_sa = 0.0f;
        int e_sq = 0;
        if (e_on) {
            e_sn = __ldg(P->s_n + e_n);
            e_sa = P->s_a[e_m];
            e_sq = gp.sumq[P->index * kGroupMaxM + e_m];
        }

        for (;;) {
            if (!mbar_wait(&full[s], ph, 4)) {
                ok = false;
                break;
            }
            const int cw = cur.chunk_words();
            unsigned char* wst = ring + s * stage_bytes;
            unsigned char* qst = wst + RT * kTileBytes;
            if (16 * warp < cw) {
                uint32_t qb[NT][4 * T::NPL];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int m = nt * 8 + g;
                    // single token: every lane reads token 0 (a broadcast); accumulator columns 1..7 then
                    // hold copies that are never read, and no lane needs predication or zero fill
                    if (M1 || m < M) {
                        const uint4* src = reinterpret_cast<const uint4*>(qst + (M1 ? 0 : m) * T::QSTRIDE + q_off);
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
                    const uint4 wa = *reinterpret_cast<const uint4*>(wst + rt * kTileBytes + a_off);
                    const uint4 wb = *reinterpret_cast<const uint4*>(wst + rt * kTileBytes + a_off + 512);
                    mma_tile_step<LV, NT, true>(acc[rt], wa, wb, qb);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
            if (++s == stages) s = 0, ph ^= 1;
            const bool last = cur.last_chunk();
            cur.next();
            if (last) break;
        }
        if (!ok) break;

        // item epilogue: one barrier; the other reduction buffer belongs to the next item
#pragma unroll
        for (int rt = 0; rt < RT; ++rt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int a = 0; a < T::NACC; ++a) {
                    int* dst = red + ((warp * RT + rt) * T::NACC + a) * 16 * M;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (M1 && (i & 1)) continue;  // token 1 does not exist
                        const int tok = nt * 8 + 2 * cq + (i & 1);
                        if (tok < M) dst[tok * 16 + g + ((i & 2) ? 8 : 0)] = acc[rt][nt][a][i];
                    }
                }
        consumer_bar_sync();
        if (e_on) {
            const int rt = e_row / 16, r = e_row % 16;
            int v[T::NACC];
#pragma unroll
            for (int a = 0; a < T::NACC; ++a) {
                int S = 0;
#pragma unroll
                for (int w = 0; w < kDecWarps; ++w) S += red[(((w * RT + rt) * T::NACC + a) * M + e_m) * 16 + r];
                v[a] = S;
            }
            const int acc_v = level_sum<LV, true, T::NACC>(v, e_sq);
            const size_t idx = static_cast<size_t>(e_m) * P->N + e_n;
            if (P->acc_debug) P->acc_debug[idx] = acc_v;
            const float y = scale_epilogue(acc_v, e_sa, e_sn);
            if (gp.y_bf16) static_cast<uint16_t*>(P->Y)[idx] = f32_to_bf16_bits(y);
            else static_cast<float*>(P->Y)[idx] = y;
        }
    }
    if (!ok) *fail = 1;
}

// ------------------------------------------------------------------------------------------------
// grouped product for 9..16 token rows
// ------------------------------------------------------------------------------------------------
// With more than eight tokens the split of a stage along K over the eight consumer warps stops paying:
// every item then ends in a cross-warp reduction of rows x tokens x 8 partial sums, as much work as
// the product itself, and its buffers leave room for two small stages only.  Here an item is 128
// rows and the warps split it by ROWS: warp w owns the 16-row tile w of the item for the whole K
// loop, accumulates all 16 tokens in registers and writes its outputs itself -- no reduction, no CTA
// barrier.  The price is that every warp reads the whole activation slice of a stage, so stages are
// half tiles (64 words per row: 32 KB of weights + 17 KB of activations at 16 tokens), four deep.
constexpr int kWideRows = 16 * kDecWarps;        // 128 rows per item with one tile per warp

// CWARPS consumer warps with RT row tiles each: an item is 16 * CWARPS * RT rows.  256-row items come either as
// sixteen warps (twice the warps to hide the latencies of the load -> logic -> product chains) or as two tiles per
// warp (the activation registers of a slice feed both tiles); their stages are a quarter tile of K (32 words) so
// that as many stages fit as with 128 rows.
// CTAs per SM of the row-split kernel.  With one token tile the PoT and the three-bit variants issue two product
// instructions and two or more logic operations per packed word where the two-bit sets issue one; two CTAs of
// half-size stages keep the pipes fed across each other's stage hand-overs (96 registers per thread is the limit for
// two CTAs of nine warps).  Measured, whole steps: three-bit codes 5.89 -> 6.61 TB/s (32 LLaMA-2-7B layers, M = 1), PoT
// 4.06 -> 4.22 (M = 1), 3.93 -> 4.04 (M = 4); the standard set 5.82 -> 5.75 at M = 4, so the two-bit sets keep one CTA
// there.  With two token tiles (9 .. 16 rows) the two-bit sets are bound by the issue of the product instructions and
// gain as well (16 LLaMA-3.1-8B layers at 16 rows: 4.07 TB/s with 256-row items on one CTA, 4.27 with two CTAs of 128-row
// items; 128 -> 96 registers without spills).
__host__ __device__ constexpr int wide_ctas_per_sm(int lv, int nt, int tiles) {
    return (((lv == QIFT_LEVELS_POT || lv == QIFT_LEVELS_INT3) && nt == 1 && tiles == 8) ||
            ((lv == QIFT_LEVELS_MNZ || lv == QIFT_LEVELS_SYM) && nt == 2 && tiles == 8)) ? 2 : 1;
}
__host__ __device__ constexpr int wide_chunk_words(int tiles, int nt, int lv = QIFT_LEVELS_MNZ) {
    // three-bit codes: a tile column is 96 bytes, not 64; two CTAs per SM: half the shared memory each
    return (tiles > 8 || nt > 2 || lv == QIFT_LEVELS_INT3 || wide_ctas_per_sm(lv, nt, tiles) > 1) ? 64 : 128;
}
__host__ __device__ constexpr int wide_token_tiles(int M) { return M > 32 ? 8 : M > 16 ? 4 : M > 8 ? 2 : 1; }

__host__ __device__ inline size_t wide_stage_bytes(int lv, int M, int tiles) {
    const int cw = wide_chunk_words(tiles, wide_token_tiles(M), lv);
    return static_cast<size_t>(tiles) * (cw * tile_word_bytes(lv)) + static_cast<size_t>(M) * (cw * codes_per_word(lv));
}
__host__ __device__ inline size_t wide_smem_bytes(int lv, int M, int tiles, int stages, int count) {
    return static_cast<size_t>(count) * sizeof(SmemProblem) + stages * (wide_stage_bytes(lv, M, tiles) + 16) + 16;
}

template <int LV, int NT, int RT, int CWARPS>
__global__ void __launch_bounds__((CWARPS + 1) * 32, wide_ctas_per_sm(LV, NT, CWARPS * RT))
linear_grouped_wide_kernel(const GroupParams gp) {
    using T = DecodeTraits<LV>;
    constexpr int TILES = CWARPS * RT;           // row tiles per item
    constexpr int CW = wide_chunk_words(TILES, NT, LV);
    constexpr int THREADS = (CWARPS + 1) * 32;
    constexpr bool INT3 = (LV == QIFT_LEVELS_INT3);
    static_assert(!INT3 || NT <= 2, "three-bit codes: six accumulator sets per token tile, at most two token tiles");
    constexpr int WB = tile_word_bytes(LV);
    // PoT with two token tiles: levels by table lookup (pot_lut_operands) instead of code bit planes -- half the
    // product instructions for more logic per word, which pays once the products are the bottleneck (measured on 16
    // LLaMA-2-7B layers: 261 against 295 us at 16 rows, but 197 against 189 us at 8).
    constexpr bool POT_LUT = (LV == QIFT_LEVELS_POT) && NT >= 2;
    constexpr int NACC = POT_LUT ? 1 : T::NACC;
    constexpr int TILE_STAGE = CW * WB;          // bytes of one tile in a stage: CW words x 16 rows, contiguous in the packed order
    constexpr int CB = CW * T::PER;              // bytes of one token's activations in a full chunk
    using Cursor = GroupCursor<T::PER, CW, WB>;
    extern __shared__ __align__(128) unsigned char smem[];
    const int M = gp.M;
    const uint32_t stage_bytes = static_cast<uint32_t>(wide_stage_bytes(LV, M, TILES));
    const int stages = gp.stages;
    unsigned char* ring = smem;
    SmemProblem* table = reinterpret_cast<SmemProblem*>(smem + stages * stage_bytes);
    uint64_t* full = reinterpret_cast<uint64_t*>(table + gp.count);
    uint64_t* empty = full + stages;
    volatile int* fail = reinterpret_cast<volatile int*>(empty + stages);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], CWARPS);
        }
        mbar_fence_init();
        *fail = 0;
    }
    for (int i = tid; i < gp.count; i += THREADS) {
        const GroupProblemDev& P = gp.use_single ? gp.single : gp.problems[i];
        SmemProblem e;
        e.packed = reinterpret_cast<const unsigned char*>(P.packed);
        e.q_a = P.q_a, e.s_n = P.s_n, e.s_a = P.s_a, e.Y = P.Y, e.acc_debug = P.acc_debug;
        e.N = P.N, e.K = P.K, e.item_begin = P.item_begin, e.index = P.quant_src;
        table[i] = e;
    }
    __syncthreads();

    if (warp == CWARPS) {
        // ---------------------------------------------------------------- producer warp
        auto expect = [&](const Cursor& c, int s) {
            if (lane == 0) mbar_expect_tx(&full[s], c.chunk_words() * (WB * c.tiles_valid + T::PER * M));
            __syncwarp();
        };
        auto issue_w = [&](const Cursor& c, int s) {  // one bulk copy per 16-row tile: the chunk's slices are contiguous in it
            const uint32_t bytes = c.chunk_words() * WB;
            unsigned char* dst = ring + s * stage_bytes;
            if (lane < c.tiles_valid)
                bulk_g2s(dst + lane * TILE_STAGE, c.wbase + lane * c.rb_bytes + static_cast<size_t>(c.chunk) * TILE_STAGE, bytes, &full[s]);
        };
        auto issue_q = [&](const Cursor& c, int s) {
            // chunk-major q_a (ChunkMajorDst): the chunk of all M tokens is one contiguous piece
            if (lane == 0)
                bulk_g2s(ring + s * stage_bytes + TILES * TILE_STAGE, c.q_a + static_cast<size_t>(c.chunk) * CB * M,
                         static_cast<uint32_t>(c.chunk_words() * T::PER * M), &full[s]);
        };
        Cursor a;
        a.init(table, gp.count, gp.item_first, gp.item_end, 16 * TILES);
        int pre = 0;
        for (; pre < stages && a.valid(); ++pre, a.next()) {  // weights do not depend on the previous kernel
            expect(a, pre);
            issue_w(a, pre);
        }
        pdl_wait();
        Cursor b;
        b.init(table, gp.count, gp.item_first, gp.item_end, 16 * TILES);
        for (int i = 0; i < pre; ++i, b.next()) issue_q(b, i);
        int s = 0;
        uint32_t ph = 0;
        for (; b.valid(); b.next()) {
            if (!mbar_wait(&empty[s], ph, 5)) break;
            expect(b, s);
            issue_w(b, s);
            issue_q(b, s);
            if (++s == stages) s = 0, ph ^= 1;
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    pdl_wait();
    const int g = lane >> 2, cq = lane & 3;
    // per-lane byte offsets inside a stage, fixed for the whole kernel
    // Activations of a stage: token after token, a token's chunk contiguous, its 16-byte groups permuted as
    // ChunkMajorDst describes.  A lane needs the NPL groups of its block per token and slice (its four packed words x
    // PER codes), block cq of the slice; it visits them in order and finds group i at swizzled_group(i).
    // Token columns beyond M read the last token's bytes: a column of the product depends on its own
    // activations only, and those columns are never written.
    int q_tok[NT];
    uint32_t q_piece[NT][T::NPL];   // byte offset inside the token's chunk of the i-th piece this lane visits
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        q_tok[nt] = min(nt * 8 + g, M - 1);
#pragma unroll
        for (int i = 0; i < T::NPL; ++i)
            q_piece[nt][i] = 16 * swizzled_group(T::NPL * cq + i, q_tok[nt], T::PER == 16);
    }
    const uint32_t ring_addr = smem_u32(ring);
    Cursor cur;
    cur.init(table, gp.count, gp.item_first, gp.item_end, 16 * TILES);
    bool ok = true;
    int s = 0;
    uint32_t ph = 0;
    while (cur.valid() && ok) {
        // With one token tile a warp would have only NACC dependent chains of product instructions; alternate
        // slices then go to a second set of accumulators (added up before the epilogue).
        constexpr int KS = (NT * RT == 1 && !INT3) ? 2 : 1;
        int acc[KS][RT][NT][NACC][4];
#pragma unroll
        for (int k = 0; k < KS; ++k)
#pragma unroll
            for (int r = 0; r < RT; ++r)
#pragma unroll
                for (int b = 0; b < NT; ++b)
#pragma unroll
                    for (int t = 0; t < NACC; ++t)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[k][r][b][t][i] = 0;
        const SmemProblem* P = &table[cur.p];
        const int cur_n0 = cur.n0;
        const int tile0 = warp * RT;                       // this warp's tiles: tile0 .. tile0 + RT - 1
        const int tiles_on = min(RT, cur.tiles_valid - tile0);   // <= 0: nothing to do in this item
        // what the epilogue needs besides the accumulators, fetched now so that the latency of these loads is
        // hidden behind the K loop instead of standing between two items
        int e_sq[NT][2];
        float e_sa[NT][2], e_sn[RT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int tok = min(nt * 8 + 2 * cq + j, M - 1);
                e_sq[nt][j] = gp.sumq[P->index * kGroupMaxM + tok];
                e_sa[nt][j] = P->s_a[tok];
            }
#pragma unroll
        for (int r = 0; r < RT; ++r)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int n = cur_n0 + 16 * (tile0 + r) + g + 8 * j;
                e_sn[r][j] = (n < P->N) ? __ldg(P->s_n + n) : 0.0f;
            }

        for (;;) {
            if (!mbar_wait(&full[s], ph, 6)) {
                ok = false;
                break;
            }
            const int cw = cur.chunk_words();
            if (tiles_on > 0) {
                // A warp whose second tile lies beyond the matrix computes it on stale bytes of the stage
                // (the copy skipped it) and drops the result in the epilogue.
                const uint32_t qs = ring_addr + s * stage_bytes + TILES * TILE_STAGE;
                const uint32_t ws = ring_addr + s * stage_bytes + tile0 * TILE_STAGE;
                uint32_t qa[NT][T::NPL];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int i = 0; i < T::NPL; ++i) qa[nt][i] = qs + q_tok[nt] * (cw * T::PER) + q_piece[nt][i];
                const uint32_t wa_base = ws + lane * 16;
                // the lane's four words of rows g and g+8 of row tile r
                auto load_words = [&](int r, int sl, uint4& wa, uint4& wb) {
                    const uint32_t o = r * TILE_STAGE + sl * (16 * WB);
                    wa = lds128(wa_base + o), wb = lds128(wa_base + o + 512);
                };
                auto slice = [&](int sl, auto ks) {
                    if constexpr (NT <= 2) {
                        uint32_t qb[NT][4 * T::NPL];
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                            for (int i = 0; i < T::NPL; ++i) {
                                const uint4 v = lds128(qa[nt][i] + sl * (16 * T::PER));
                                qb[nt][4 * i] = v.x, qb[nt][4 * i + 1] = v.y, qb[nt][4 * i + 2] = v.z, qb[nt][4 * i + 3] = v.w;
                            }
                        }
#pragma unroll
                        for (int r = 0; r < RT; ++r) {
                            uint4 wa, wb;
                            load_words(r, sl, wa, wb);
                            if constexpr (INT3) {   // the lane's high words follow the slice's two groups of low words
                                const uint4 wh = lds128(wa_base + r * TILE_STAGE + sl * (16 * WB) + 1024);
                                mma_tile_step_int3<NT>(acc[decltype(ks)::value][r], wa, wb, wh, qb);
                            } else if constexpr (POT_LUT) mma_tile_step_pot_lut<NT>(acc[decltype(ks)::value][r], wa, wb, qb);
                            else mma_tile_step<LV, NT, true>(acc[decltype(ks)::value][r], wa, wb, qb);
                        }
                    } else {
                        // many token tiles: the activation words are fetched as they are used (all of them would not
                        // fit the registers); piece i of a token tile serves 4 / NPL packed words
                        static_assert(RT == 1, "one row tile per warp with more than two token tiles");
                        uint4 wa, wb;
                        load_words(0, sl, wa, wb);
                        const uint32_t lo[4] = {wa.x, wa.y, wa.z, wa.w};
                        const uint32_t hi[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                        for (int i = 0; i < T::NPL; ++i) {
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                const uint4 v = lds128(qa[nt][i] + sl * (16 * T::PER));
                                const uint32_t q4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                                for (int j = 0; j < 4 / T::NPL; ++j) {   // the words this piece belongs to
                                    const int word = i * (4 / T::NPL) + j;
                                    uint32_t qw[T::NPL];
#pragma unroll
                                    for (int t = 0; t < T::NPL; ++t) qw[t] = q4[j * T::NPL + t];
                                    mma_word<LV, POT_LUT, NACC>(acc[0][0][nt], lo[word], hi[word], qw);
                                }
                            }
                        }
                    }
                };
                if (cw == CW) {
#pragma unroll
                    for (int sl = 0; sl < CW / 16; sl += 2) {
                        slice(sl, std::integral_constant<int, 0>{});
                        slice(sl + 1, std::integral_constant<int, KS - 1>{});
                    }
                } else {
                    for (int sl = 0; 16 * sl < cw; ++sl) slice(sl, std::integral_constant<int, 0>{});   // 16-word slices of a short last chunk
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
            if (++s == stages) s = 0, ph ^= 1;
            const bool last = cur.last_chunk();
            cur.next();
            if (last) break;
        }
        if (!ok) break;

        if (KS == 2) {
#pragma unroll
            for (int r = 0; r < RT; ++r)
#pragma unroll
                for (int b = 0; b < NT; ++b)
#pragma unroll
                    for (int t = 0; t < NACC; ++t)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[0][r][b][t][i] += acc[KS - 1][r][b][t][i];
        }
        // epilogue from registers: rows g and g+8 of each tile, tokens nt*8 + 2cq + {0,1}; the scales and token
        // sums were fetched when the item began
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            if (r >= tiles_on) continue;
            const int row0 = cur_n0 + 16 * (tile0 + r);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tok = nt * 8 + 2 * cq + (i & 1);
                    const int n = row0 + g + ((i & 2) ? 8 : 0);
                    if (tok < M && n < P->N) {
                        int acc_v;
                        if constexpr (POT_LUT) {
                            acc_v = acc[0][r][nt][0][i];   // the operands were the levels themselves
                        } else {
                            int v[NACC];
#pragma unroll
                            for (int a = 0; a < NACC; ++a) v[a] = acc[0][r][nt][a][i];
                            acc_v = level_sum<LV, true, NACC>(v, e_sq[nt][i & 1]);
                        }
                        const size_t idx = static_cast<size_t>(tok) * P->N + n;
                        if (P->acc_debug) P->acc_debug[idx] = acc_v;
                        const float y = scale_epilogue(acc_v, e_sa[nt][i & 1], e_sn[r][i >> 1]);
                        if (gp.y_bf16) static_cast<uint16_t*>(P->Y)[idx] = f32_to_bf16_bits(y);
                        else static_cast<float*>(P->Y)[idx] = y;
                    }
                }
        }
    }
    if (!ok) *fail = 1;
}

}  // namespace qift

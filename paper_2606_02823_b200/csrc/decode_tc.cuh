// Weight-streaming product for 9 .. 128 token rows on the tcgen05 tensor cores (the two-bit sets and INT4).
//
// With more than eight token rows the mma.sync decode kernels are bound by the issue rate of the legacy tensor
// instructions and by shared-memory reads of the activations, not by HBM.  Here the roles of the operands are
// swapped: the 128 output channels of a work item are the M side of tcgen05.mma (kind::i8, cta_group::1), the
// token rows its N side (16 .. 128), and the packed codes become the A operand IN TENSOR MEMORY -- they never
// exist as int8 in shared memory, which a path that streams weights at the HBM rate could not afford (four
// times the packed bytes written and read again).
//
//   warp 0      activation producer: per 128-byte k-block the q_a rows of all tokens, one tensor copy (TMA, no
//               multicast) into a 128-byte-swizzled K-major stage (the B operand)
//   warp 1      tensor-memory allocation, tcgen05.mma issue: D[128 channels x tokens] += A(tmem) * B(smem)
//   warp 14     second issuer.  A thread issues a tcgen05 instruction every ~50 cycles at best (the measured 26 ns per
//               128 x N x 32 instruction for N <= 64 is this issue cost, not tensor time), so the (k-block, tile) units are
//               dealt alternately to two threads.  Integer accumulation commutes and every instruction accumulates
//               (the epilogue leaves the accumulator columns zeroed), so the two streams need no order between them.
//   warps 2-5, 15-18   epilogue, two warps per tensor-memory lane quarter on alternate 16-token chunks: tcgen05.ld
//               (lane = channel, column = token), level map with the token sums, the two scale multiplies, stores (a
//               warp's 32 lanes write 32 consecutive channels of a token row), zeros written back to the columns read
//   warps 6-13  expanders, two per tensor-memory lane quarter (alternate 16-word slices): each streams the packed
//               words of ITS 32 channel rows with cp.async into a private shared-memory ring (16-byte chunks XOR-swizzled by row:
//               conflict-free 128-bit reads; up to eight 2 KB units in flight per warp, running ahead across items), turns
//               a packed word into operand words with one logic operation each (plus one shift per two-bit word) and
//               writes 32 columns per k-block with tcgen05.st into an eight-deep operand ring in tensor memory
// An item is R = 1, 2 or 4 blocks of 128 channels: the activations of a k-block are staged once for all of them.
// Operand bytes are the stored codes times a place value (two-bit: planes 0 / 2 times 1, planes 1 / 3 times 4;
// INT4: nibble ^ 8 times 1 / 16); the activations come PRESCALED (bytes of the even planes hold 4 q, INT4: plane
// 0 holds 16 q), so every product carries the same factor (4 or 16), which an arithmetic shift removes exactly;
// the affine level map is undone with sum_k q as everywhere else.  PoT is not affine in the code: its operand bytes are
// the levels themselves (byte-permute table lookup, a signed A operand) against unscaled activations whose bytes the
// quantizer wrote in the matching order.  The accumulators (R blocks x tokens <= 128
// columns) are double-buffered in tensor memory: 2 x 128 columns + 8 x 32 operand columns = all 512.
// Work items (problem, 128-channel block) are dealt round-robin to one persistent CTA per SM, as in the other
// grouped kernels.  Every wait is bounded; no TMA multicast.
#pragma once

#include "common.cuh"
#include "grouped.cuh"
#include "prefill.cuh"

namespace qift {

constexpr int kTcRows = 128;       // channels per work item
constexpr int kTcExpanders = 8;    // expander warps: two per tensor-memory lane quarter
constexpr int kTcIssuers = 2;     // threads that issue tensor-core instructions (warp 1 and warp 14)
constexpr int kTcEpiGroups = 2;   // epilogue warps per tensor-memory lane quarter (warps 2-5 and 15-18), alternate 16-token chunks
constexpr int kTcThreads = 32 * (6 + kTcExpanders + (kTcIssuers - 1) + 4 * (kTcEpiGroups - 1));
constexpr int kTcSlotBytes = 32 * 64;   // a packed unit: 32 rows x 64 bytes, 16-byte chunks XOR-swizzled by row
// packed units in flight per expander warp (what is left of shared memory beside the activation ring)
__host__ __device__ constexpr int tc_wslots(int ntok) { return ntok <= 32 ? 8 : ntok <= 64 ? 6 : 4; }
constexpr int kTcARing = 8;        // k-blocks of operand columns in tensor memory
constexpr int kTcACol0 = 256;      // first operand column (columns 0 .. 255: two accumulators)
constexpr int kTcMaxM = 128;

__host__ __device__ constexpr int tc_act_stages(int ntok) { return ntok >= 128 ? 6 : 10; }
// 128-channel blocks per work item.  A slice of an item fills KPS * R slots of the operand ring (KPS = k-blocks per
// 16-word slice: 2 for two-bit codes, 1 for INT4) and the two expander warps of a lane quarter take alternate slices;
// with KPS * R <= 4 the eight ring slots return to the same warp every time, so a warp is never more than one use of a
// slot ahead of its release barrier (a parity wait cannot tell two uses apart).
__host__ __device__ constexpr int tc_tiles_per_item(int ntok, int per) {
    return per == 16 ? (ntok <= 64 ? 2 : 1) : (ntok <= 32 ? 4 : ntok <= 64 ? 2 : 1);
}
// Accumulator sets per channel block: the four tensor-core steps of a k-block go to set (step mod S), so that consecutive
// instructions do not wait for one another through one accumulator; the epilogue adds the sets (exact in INT32).
__host__ __device__ constexpr int tc_acc_sets(int ntok, int r) {
    return 128 / (r * ntok) >= 4 ? 4 : 128 / (r * ntok) >= 2 ? 2 : 1;
}
__host__ __device__ inline size_t tc_smem_bytes(int ntok, int count) {
    return 1024 + static_cast<size_t>(tc_act_stages(ntok)) * ntok * 128 + kTcExpanders * tc_wslots(ntok) * kTcSlotBytes +
           static_cast<size_t>(count) * sizeof(SmemProblem) + 512;
}

__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]),
        "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]),
        "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tc_zero16(uint32_t taddr) {   // sixteen columns of the warp's 32 lanes <- 0
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(taddr), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
          "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor]
__device__ __forceinline__ void tc_mma_i8_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Operand words of one k-block (128 codes) of a channel row.
template <int LV>
__device__ __forceinline__ void tc_operands(const uint32_t* w, uint32_t (&o)[32]) {
    if constexpr (LV == QIFT_LEVELS_POT) {   // 8 words of 16 two-bit codes: the levels themselves, by table lookup
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t a[4];
            pot_lut_operands(w[i], a);
            o[4 * i] = a[0], o[4 * i + 1] = a[1], o[4 * i + 2] = a[2], o[4 * i + 3] = a[3];
        }
    } else if constexpr (LV == QIFT_LEVELS_INT4) {  // 16 words of 8 nibbles
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            o[2 * i] = (w[i] ^ 0x88888888u) & 0x0f0f0f0fu;
            o[2 * i + 1] = (w[i] ^ 0x88888888u) & 0xf0f0f0f0u;
        }
    } else {  // 8 words of 16 two-bit codes
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t s = w[i] >> 4;
            o[4 * i] = w[i] & 0x03030303u;
            o[4 * i + 1] = w[i] & 0x0c0c0c0cu;
            o[4 * i + 2] = s & 0x03030303u;
            o[4 * i + 3] = s & 0x0c0c0c0cu;
        }
    }
}

template <int LV>
__device__ __forceinline__ int tc_level_sum(int d, int sq) {
    if constexpr (LV == QIFT_LEVELS_POT) return d;   // the operands were the levels, the activations unscaled
    if constexpr (LV == QIFT_LEVELS_MNZ) return 2 * (d >> 2) - 3 * sq;
    if constexpr (LV == QIFT_LEVELS_SYM) return (d >> 2) - 2 * sq;
    return (d >> 4) - 8 * sq;  // INT4
}

// R: 128-channel tiles per work item.  The activations of a k-block are staged once and multiplied with the R weight
// tiles of the item, which divides both the L2 traffic of the activations and the depth their ring needs by R.
// 2 R NTOK <= 256 accumulator columns.
template <int LV, int NTOK, int R>
__global__ void __launch_bounds__(kTcThreads, 1)
linear_tc_kernel(const GroupParams gp) {
    constexpr int PER = codes_per_word(LV);
    constexpr int KPS = (PER == 16) ? 2 : 1;          // k-blocks per 16-word slice
    constexpr int ASTAGES = tc_act_stages(NTOK);
    constexpr uint32_t ACT_BYTES = NTOK * 128;
    constexpr int S = tc_acc_sets(NTOK, R);           // accumulator sets per channel block
    constexpr int DBUF = R * S * NTOK;                // accumulator columns of an item
    constexpr int kTcWSlots = tc_wslots(NTOK);
    static_assert(2 * DBUF <= kTcACol0, "two accumulator buffers fit below the operand ring");
    static_assert(KPS * R <= 4, "a ring slot must always return to the same expander warp");
    // D = s32, A = u8 (operand bytes from tensor memory; PoT: s8, the levels), B = s8 (activations), both K-major, N = NTOK, M = 128
    constexpr uint32_t IDESC = (2u << 4) | ((LV == QIFT_LEVELS_POT ? 1u : 0u) << 7) | (1u << 10) | (static_cast<uint32_t>(NTOK >> 3) << 17) |
                               (static_cast<uint32_t>(kTcRows >> 4) << 24);
    using Cursor = GroupCursor<PER, 16>;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* act = smem;
    unsigned char* wring = act + ASTAGES * ACT_BYTES;
    SmemProblem* table = reinterpret_cast<SmemProblem*>(wring + kTcExpanders * kTcWSlots * kTcSlotBytes);
    uint64_t* act_full = reinterpret_cast<uint64_t*>(table + gp.count);
    uint64_t* act_empty = act_full + ASTAGES;
    uint64_t* a_full = act_empty + ASTAGES;
    uint64_t* a_empty = a_full + kTcARing;
    uint64_t* d_full = a_empty + kTcARing;
    uint64_t* d_empty = d_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(d_empty + 2);
    volatile int* fail = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = gp.M;

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < ASTAGES; ++s) {
            mbar_init(&act_full[s], 1);
            mbar_init(&act_empty[s], R < kTcIssuers ? R : kTcIssuers);   // tcgen05.commit of every issuer with a unit in the k-block
        }
        for (int s = 0; s < kTcARing; ++s) {
            mbar_init(&a_full[s], 4);   // one arrival per lane quarter
            mbar_init(&a_empty[s], 1);  // tcgen05.commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&d_full[b], kTcIssuers);
            mbar_init(&d_empty[b], 4 * kTcEpiGroups);  // the epilogue warps
        }
        *fail = 0;
        mbar_fence_init();
    }
    for (int i = tid; i < gp.count; i += kTcThreads) {
        const GroupProblemDev& P = gp.use_single ? gp.single : gp.problems[i];
        SmemProblem e;
        e.packed = reinterpret_cast<const unsigned char*>(P.packed);
        e.q_a = P.q_a, e.s_n = P.s_n, e.s_a = P.s_a, e.Y = P.Y, e.acc_debug = P.acc_debug;
        e.N = P.N, e.K = P.K, e.item_begin = P.item_begin, e.index = P.quant_src;
        table[i] = e;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ activation producer
        // One tensor copy per k-block: the plan's map of the problem's q_a [M, K], box = 128 bytes of K x NTOK token rows
        // (rows beyond M arrive as zeros), written in the 128-byte-swizzled K-major order the B descriptor reads.
        pdl_wait();
        if (lane == 0) {
            Cursor c;
            c.init(table, gp.count, gp.item_first, gp.item_end, R * kTcRows);
            uint32_t it = 0;
            bool ok = true;
            for (; c.valid() && ok; c.next()) {        // one cursor step = one slice = KPS k-blocks
                for (int j = 0; j < KPS; ++j, ++it) {
                    const int s = it % ASTAGES;
                    if (it >= static_cast<uint32_t>(ASTAGES) && !mbar_wait(&act_empty[s], ((it / ASTAGES) - 1) & 1, 60)) {
                        *fail = 1, ok = false;
                        break;
                    }
                    mbar_expect_tx(&act_full[s], ACT_BYTES);
                    tma_load_2d(act + s * ACT_BYTES, &gp.maps[c.p], (c.chunk * KPS + j) * 128, 0, &act_full[s]);
                }
            }
        }
    } else if (warp == 1 || (warp >= 6 + kTcExpanders && warp < 6 + kTcExpanders + kTcIssuers - 1)) {
        // ------------------------------------------------------------------ MMA issuers
        // Unit u = (k-block, tile) in running order goes to issuer u mod 2: with two tiles per item each issuer owns a
        // tile, with one it takes every other k-block.  One thread per issuer; the loop is kept short (a lone thread
        // retires a dependent instruction every few cycles).
        if (lane == 0) {
            const uint32_t me = (warp == 1) ? 0u : static_cast<uint32_t>(warp - (6 + kTcExpanders) + 1);
            Cursor c;
            c.init(table, gp.count, gp.item_first, gp.item_end, R * kTcRows);
            uint32_t icount = 0, it = 0;        // items, k-blocks (running)
            uint32_t sb = 0, sb_par = 0;        // activation stage of the next k-block, parity of its fill
            uint32_t slot = 0, slot_par = 0;    // operand-ring slot of the next k-block's first tile (R divides the ring), parity
            const uint64_t desc0 = make_kmajor_sw128_desc(smem_u32(act));
            bool ok = true;
            while (c.valid() && ok) {
                const int buf = icount & 1;
                if (!mbar_wait(&d_empty[buf], (icount >> 1) & 1, 61)) {   // zeroed by the epilogue (first use: at start)
                    *fail = 1;
                    break;
                }
                tc_fence_after();
                const int kblocks = c.nchunks * KPS;
                const int tiles = (c.tiles_valid + 7) >> 3;   // 128-channel tiles of the item that exist
                const uint32_t d_base = tmem_base + buf * DBUF;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    bool any = false;
                    uint64_t bdesc = 0;
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        if (((it * R + r) & (kTcIssuers - 1)) != me) continue;   // unit (k-block, tile) -> issuer, round robin
                        if (!any) {
                            if (!mbar_wait(&act_full[sb], sb_par, 63)) {
                                *fail = 1, ok = false;
                                break;
                            }
                            bdesc = desc0 + sb * (ACT_BYTES >> 4);
                            any = true;
                        }
                        if (!mbar_wait(&a_full[slot + r], slot_par, 62)) {
                            *fail = 1, ok = false;
                            break;
                        }
                        tc_fence_after();
                        if (r < tiles) {
                            const uint32_t a_base = tmem_base + kTcACol0 + (slot + r) * 32;
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4)
                                tc_mma_i8_ts(d_base + (r * S + (k4 % S)) * NTOK, a_base + 8 * k4, bdesc + 2 * k4, IDESC, 1u);
                        }
                        tc_commit(&a_empty[slot + r]);
                    }
                    if (!ok) break;
                    if (any) tc_commit(&act_empty[sb]);
                    if (++sb == ASTAGES) sb = 0, sb_par ^= 1;
                    slot += R;
                    if (slot == kTcARing) slot = 0, slot_par ^= 1;
                }
                if (!ok) break;
                tc_commit(&d_full[buf]);
                ++icount;
                c.next_item();
            }
        }
    } else if (warp < 6 || warp >= 6 + kTcExpanders + kTcIssuers - 1) {
        // ------------------------------------------------------------------ epilogue warps
        const int eg = (warp < 6) ? 0 : 1;   // this warp's 16-token chunks: eg, eg + kTcEpiGroups, ...
        const int quarter = warp & 3;
        // every tensor-core instruction accumulates: both accumulator buffers start zeroed, and each is zeroed again by
        // the warp that has read it
        auto zero_acc = [&](int buf) {   // the chunks this warp reads, in every accumulator set of every tile
#pragma unroll
            for (int col = 0; col < R * S * NTOK; col += NTOK)
                for (int m0 = 16 * eg; m0 < NTOK; m0 += 16 * kTcEpiGroups)
                    tc_zero16(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * DBUF + col + m0);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&d_empty[buf]);
        };
        zero_acc(0);
        zero_acc(1);
        pdl_wait();
        Cursor c;
        c.init(table, gp.count, gp.item_first, gp.item_end, R * kTcRows);
        uint32_t icount = 0;
        while (c.valid()) {
            const SmemProblem& P = table[c.p];
            const int buf = icount & 1;
            const int* sumq = gp.sumq + static_cast<size_t>(P.index) * kGroupMaxM;
            if (!mbar_wait(&d_full[buf], (icount >> 1) & 1, 64)) {
                *fail = 1;
                break;
            }
            tc_fence_after();
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int n = c.n0 + r * kTcRows + quarter * 32 + lane;
                if (c.n0 + r * kTcRows >= P.N) break;   // (uniform) this tile of the item does not exist
                const float sn = (n < P.N) ? __ldg(P.s_n + n) : 0.0f;
                for (int m0 = 16 * eg; m0 < M; m0 += 16 * kTcEpiGroups) {
                    uint32_t v[16];
                    tc_ld16(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * DBUF + r * S * NTOK + m0, v);
                    // the token sums and token scales of these sixteen rows, fetched while the accumulators are on their way
                    int sq[16];
                    float sa[16];
                    if (m0 + 16 <= M) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int4 a = __ldg(reinterpret_cast<const int4*>(sumq + m0) + j);
                            const float4 b = __ldg(reinterpret_cast<const float4*>(P.s_a + m0) + j);
                            sq[4 * j] = a.x, sq[4 * j + 1] = a.y, sq[4 * j + 2] = a.z, sq[4 * j + 3] = a.w;
                            sa[4 * j] = b.x, sa[4 * j + 1] = b.y, sa[4 * j + 2] = b.z, sa[4 * j + 3] = b.w;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int m = min(m0 + j, M - 1);
                            sq[j] = __ldg(sumq + m), sa[j] = __ldg(P.s_a + m);
                        }
                    }
                    tc_wait_ld();
#pragma unroll
                    for (int st = 1; st < S; ++st) {
                        uint32_t u[16];
                        tc_ld16(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * DBUF + (r * S + st) * NTOK + m0, u);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] += u[j];
                    }
                    if (n < P.N) {
                        size_t o = static_cast<size_t>(m0) * P.N + n;
#pragma unroll
                        for (int j = 0; j < 16; ++j, o += P.N) {
                            if (m0 + j < M) {
                                const int acc = tc_level_sum<LV>(static_cast<int>(v[j]), sq[j]);
                                const float y = scale_epilogue(acc, sa[j], sn);
                                if (gp.y_bf16) static_cast<uint16_t*>(P.Y)[o] = f32_to_bf16_bits(y);
                                else static_cast<float*>(P.Y)[o] = y;
                                if (P.acc_debug) P.acc_debug[o] = acc;
                            }
                        }
                    }
                }
            }
            zero_acc(buf);
            ++icount;
            c.next_item();
        }
    } else if (warp < 6 + kTcExpanders) {
        // ------------------------------------------------------------------ expander warps
        // Two warps per lane quarter; warp (q, ph) takes the slices whose running number has parity ph.  A unit =
        // one slice of one tile of the item (its 32 rows x 64 bytes); units are fetched kTcWSlots ahead.
        const int e = warp - 6, q = warp & 3, ph = e >> 2;   // q: the lane quarter this warp's tcgen05.st can reach
        const uint32_t ring_u32 = smem_u32(wring + e * kTcWSlots * kTcSlotBytes);
        Cursor f, c;
        f.init(table, gp.count, gp.item_first, gp.item_end, R * kTcRows);
        c.init(table, gp.count, gp.item_first, gp.item_end, R * kTcRows);
        uint32_t fg = 0, fr = 0;                    // fetch side: running slice number, next tile of the slice
        auto fetch = [&](int slot) {                // the next own unit -> ring slot; always commits a group
            while (f.valid() && (fg & 1) != static_cast<uint32_t>(ph)) f.next(), ++fg;
            if (f.valid()) {
                const unsigned char* base = f.wbase + static_cast<size_t>(f.chunk >> 3) * kTileBytes + (f.chunk & 7) * 1024 + lane * 16;
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const int rb = 8 * static_cast<int>(fr) + 2 * q + (h >> 1);
                    if (rb < f.tiles_valid)
                        cp_async16(ring_u32 + slot * kTcSlotBytes + (h * 8 + (lane >> 2)) * 64 + (((lane & 3) ^ ((lane >> 3) & 3)) << 4),
                                   base + rb * f.rb_bytes + (h & 1) * 512);   // row h * 8 + lane / 4: chunk ^ ((row >> 1) & 3)
                }
                if (++fr == R) fr = 0, f.next(), ++fg;
            }
            cp_async_commit();
        };
        for (int s = 0; s < kTcWSlots; ++s) fetch(s);
        uint32_t g = 0, kbc = 0, units = 0;         // running slice number, k-blocks before this slice, units consumed
        bool ok = true;
        for (; c.valid() && ok; c.next(), ++g, kbc += KPS) {
            if ((g & 1) != static_cast<uint32_t>(ph)) continue;
#pragma unroll
            for (int r = 0; r < R; ++r, ++units) {
                const int slot = units % kTcWSlots;
                cp_async_wait<kTcWSlots - 1>();     // the oldest group = this unit
                __syncwarp();
                const bool row_valid = (8 * r + 2 * q + (lane >> 4)) < c.tiles_valid;
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (row_valid) v = lds128(ring_u32 + slot * kTcSlotBytes + lane * 64 + ((i ^ ((lane >> 1) & 3)) << 4));
                    w[4 * i] = v.x, w[4 * i + 1] = v.y, w[4 * i + 2] = v.z, w[4 * i + 3] = v.w;
                }
                __syncwarp();                       // every lane has read the slot before it is refilled
                fetch(slot);
#pragma unroll
                for (int j = 0; j < KPS; ++j) {
                    const uint32_t ia = (kbc + j) * R + r;
                    const int sa = ia % kTcARing;
                    if (ia >= static_cast<uint32_t>(kTcARing) && !mbar_wait(&a_empty[sa], ((ia / kTcARing) - 1) & 1, 65)) {
                        *fail = 1, ok = false;
                        break;
                    }
                    tc_fence_after();
                    uint32_t o[32];
                    tc_operands<LV>(w + (PER == 16 ? 8 * j : 0), o);
                    tc_st32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + kTcACol0 + sa * 32, o);
                }
                if (!ok) break;
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < KPS; ++j) mbar_arrive(&a_full[((kbc + j) * R + r) % kTcARing]);
                }
            }
        }
        cp_async_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

}  // namespace qift

// Shared device helpers of the qift CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qift.h"

namespace qift {

// ------------------------------------------------------------------------------------------------
// Device status word: a kernel whose bounded wait expires records (site | block << 8) here and
// returns normally; qift_device_status() reads and clears it.
// ------------------------------------------------------------------------------------------------
static __device__ unsigned int g_status_word;

__device__ __forceinline__ void report_timeout(unsigned int site) {
    atomicCAS(&g_status_word, 0u, (site & 0xffu) | (blockIdx.x << 8) | 0x80000000u);
}

// ------------------------------------------------------------------------------------------------
// Level sets
// ------------------------------------------------------------------------------------------------
__host__ __device__ constexpr int codes_per_word(int lv) { return lv == QIFT_LEVELS_INT4 ? 8 : 16; }
__host__ __device__ constexpr float top_level(int lv) {
    return lv == QIFT_LEVELS_MNZ ? 3.0f : lv == QIFT_LEVELS_POT ? 4.0f : lv == QIFT_LEVELS_SYM ? 1.0f : lv == QIFT_LEVELS_INT3 ? 3.0f : 7.0f;
}

// ------------------------------------------------------------------------------------------------
// Packed-weight storage order.  Words live in tiles of 16 rows x 128 words (the last tile of a row
// block may be narrower), row blocks outermost.  Inside a tile, 16-byte groups of four consecutive
// words of one row are ordered (slice = word/16, half = row/8, row%8, quad = word/4 % 4): the 32
// groups a warp needs for one mma step (8 rows x 4 quads) are 512 contiguous bytes, so a tile is
// one bulk copy and every shared-memory read of it is a conflict-free 128-bit access.  Rows and
// words per row are padded to multiples of 16 with zero words.
// ------------------------------------------------------------------------------------------------
constexpr int kTileRows = 16;
constexpr int kChunkWords = 128;                               // words per row in a full tile
constexpr int kTileBytes = kTileRows * kChunkWords * 4;        // 8192

__host__ __device__ constexpr int round_up16(int v) { return (v + 15) & ~15; }
__host__ __device__ inline int packed_pitch(int K, int lv) { return round_up16(K / codes_per_word(lv)); }
__host__ __device__ inline size_t packed_word_address(int n, int j, int pitch) {
    const int rb = n >> 4, half = (n >> 3) & 1, g = n & 7;
    const int c = j >> 7, jj = j & 127;
    const int slice = jj >> 4, quad = (jj >> 2) & 3, e = jj & 3;
    return static_cast<size_t>(rb) * 16 * pitch + static_cast<size_t>(c) * (kTileRows * kChunkWords) +
           static_cast<size_t>((((slice * 2 + half) * 32 + g * 4 + quad) << 2) + e);
}

// Three-bit codes (INT3): a two-bit plane in words as above and a one-bit plane, 32 codes to a word, interleaved
// slice by slice.  A slice -- 16 low words of the 16 rows of a row block -- is 1536 contiguous bytes: 1024 of low
// words in the group order above (rows 0..7, then rows 8..15), then 512 of high words, group (row%8)*4 + quad holding
// {high words 0, 1 of row row%8, high words 0, 1 of row row%8 + 8} of that quad: the 16 bytes a lane of the product
// kernel needs next to its two groups of low words.  High word h of a row covers low words 2h, 2h+1; the bit of
// code k = 16j + 4t + b is bit 8b + 4(j%2) + {0,2,1,3}[t].  Row blocks are 24 * pitch words (pitch = low words per
// row, padded to 16).
__host__ __device__ constexpr int tile_word_bytes(int lv) { return lv == QIFT_LEVELS_INT3 ? 96 : 64; }   // 16 rows x one low word
__host__ __device__ inline size_t int3_low_address(int n, int j, int pitch) {
    const int rb = n >> 4, half = (n >> 3) & 1, g = n & 7;
    const int slice = j >> 4, quad = (j >> 2) & 3, e = j & 3;
    return static_cast<size_t>(rb) * 24 * pitch + static_cast<size_t>(slice) * 384 + static_cast<size_t>(((half * 32 + g * 4 + quad) << 2) + e);
}
__host__ __device__ inline size_t int3_high_address(int n, int j, int pitch) {   // j: low word index
    const int rb = n >> 4, half = (n >> 3) & 1, g = n & 7;
    const int slice = j >> 4, quad = (j >> 2) & 3, pair = (j >> 1) & 1;
    return static_cast<size_t>(rb) * 24 * pitch + static_cast<size_t>(slice) * 384 + 256 + static_cast<size_t>(((g * 4 + quad) << 2) + 2 * half + pair);
}
__host__ __device__ constexpr int int3_high_shift(int j, int t) { return 4 * (j & 1) + ((t & 1) << 1) + (t >> 1); }   // inside a byte
// Four level bytes of plane t of low word `lo` (index j) and its high word `hi`: (c & 3) - 4 (c >> 2) = (c & 3) | 0xfc [c >> 2].
__device__ __forceinline__ uint32_t int3_level_bytes(uint32_t lo, uint32_t hi, int j, int t) {
    return ((lo >> (2 * t)) & 0x03030303u) | (((hi >> int3_high_shift(j, t)) & 0x01010101u) * 0xfcu);
}

template <int LV>
__device__ __forceinline__ int level_from_code(int c) {
    if constexpr (LV == QIFT_LEVELS_INT3) return ((c & 7) ^ 4) - 4;
    if constexpr (LV == QIFT_LEVELS_MNZ) return 2 * c - 3;
    if constexpr (LV == QIFT_LEVELS_POT) return 3 * c - (c >> 1) - 4;  // 0,3,5,8 minus 4
    if constexpr (LV == QIFT_LEVELS_SYM) return c - 2;
    return ((c & 15) ^ 8) - 8;
}

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Programmatic dependent launch: let the next kernel in the stream start its prologue, and wait for
// the previous kernel's memory before touching any caller buffer.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)  // time hint: the hardware may park the thread while it waits
        : "memory");
    return ok != 0;
}
// thread-block clusters
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: polls (each poll may be parked by the hardware for up to its time hint) until the
// phase completes or `limit_ns` of wall time have passed (two seconds unless the launch says otherwise);
// then records the site and returns false.  Callers skip their remaining work on false.
constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, unsigned int site, uint64_t limit_ns = kWaitLimitNs) {
    uint64_t t0 = 0;
    const uint32_t hint = limit_ns < 1000000ull ? static_cast<uint32_t>(limit_ns) : 1000000u;
    for (;;) {
        if (mbar_try_wait(bar, parity, hint)) return true;
        const uint64_t t = global_timer_ns();
        if (t0 == 0) t0 = t;
        else if (t - t0 > limit_ns) break;
    }
    report_timeout(site);
    return false;
}

// 1-D bulk copy global -> shared::cta (no multicast), completion counted on an mbarrier.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Shared-memory loads by 32-bit shared address: the address arithmetic stays 32-bit and a constant
// displacement folds into the instruction.
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

// u8 x s8 -> s32 four-way dot product.
__device__ __forceinline__ int dp4a_us(uint32_t a_u8x4, uint32_t b_s8x4, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a_u8x4), "r"(b_s8x4), "r"(c));
    return d;
}

// D(16x8,s32) += A(16x32,u8,row) * B(32x8,s8,col)
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// D(16x8,s32) += A(16x32,s8,row) * B(32x8,s8,col)
__device__ __forceinline__ void mma_s8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint16_t f32_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// y = ((float)acc * s_a) * s_n, two separately rounded multiplies.
__device__ __forceinline__ float scale_epilogue(int acc, float s_a, float s_n) {
    return __fmul_rn(__fmul_rn(static_cast<float>(acc), s_a), s_n);
}

}  // namespace qift

// Prefill product on CTA pairs with the code expansion fused in: no N*K scratch, no expansion pass.
//
// gemm_i8_pair_kernel is bound by what an SM can pull from L2 (per 128-byte k-block 16 KB of
// activations + 16 KB of expanded weights for 128 x 256 x 128 MACs) and needs a separate pass that
// writes N*K bytes of int8 levels.  Here each CTA of a pair still TMA-loads its own 128 tokens, but
// its half of the weight tile comes in as PACKED codes (4 KB per k-block for 2-bit weights): the
// producer warp bulk-copies them slice by slice (16 words per row: 1 KB per 16-row block, contiguous in
// the tiled layout) into a small shared-memory ring; eight expander warps read them from there, turn
// each word into unsigned byte operand words (one shift + one mask per four codes) and store them
// into the 128-byte-swizzled stage.  (Loading the packed words with ordinary global loads held in
// registers does not work here: the release that publishes a finished stage waits for every global
// load the thread has in flight, which serialises the prefetch.)  tcgen05.mma.cta_group::2 (kind::i8, A = s8 activations, B = u8 codes) multiplies; the affine
// level map is undone in the epilogue with the per-token sum of q_a.  Because a CTA expands only half
// of the tile's channels for 128 tokens x the full tile width of MACs, the expanders have 512 tensor
// clocks per k-block for 16 KB of operand bytes (the single-CTA fused kernel has 256 for 32 KB).
//
//   warp 0      TMA producer for this CTA's activation tile
//   warp 1      tensor-memory allocation; in the leader CTA, tcgen05.mma issue for the pair
//   warps 2-5   epilogue (tcgen05.ld, level map, scales, stores)
//   warps 6-13  expanders
// A stage is full when the leader's barrier has seen both CTAs' activation bytes and one arrival per
// expander warp of BOTH CTAs; the peer's expanders arrive with release semantics at cluster scope
// after a proxy fence, and the leader's MMA thread acquires at cluster scope, so the generic-proxy
// stores of either CTA are visible to the tensor core.  No TMA multicast.  Every wait is bounded.
#pragma once

#include "common.cuh"
#include "prefill.cuh"
#include "prefill_2cta.cuh"
#include "prefill_fused.cuh"

namespace qift {

constexpr int kFusedPairStages = 6;
constexpr int kExpanderGroups = 2;  // expander warps are split into groups that take alternate packed slices
constexpr int kGroupWarps = kFusedExpanderWarps / kExpanderGroups;
constexpr int kPackedSlots = 4;  // ring of packed slices (16 words per row, at most 128 rows: 8 KB each)

__device__ __forceinline__ void mbar_arrive_leader_release(uint64_t* bar) {  // same offset in CTA rank 0, release at cluster scope
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(smem_u32(bar) & kPeerBitMask) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, unsigned int site) {
    uint64_t t0 = 0;
    for (;;) {
        if (mbar_try_wait_cluster(bar, parity, 1000000u)) return true;
        const uint64_t t = global_timer_ns();
        if (t0 == 0) t0 = t;
        else if (t - t0 > kWaitLimitNs) break;
    }
    report_timeout(site);
    return false;
}

template <int BN>
__host__ __device__ constexpr size_t fused_pair_smem_bytes() {
    return 1024 + static_cast<size_t>(kFusedPairStages) * (kGemmBM * kGemmBK + (BN / 2) * kGemmBK) +
           static_cast<size_t>(kPackedSlots) * (BN / 2) * 64 + 256;
}

template <int LV, int BN>
__global__ void __launch_bounds__(kFusedThreads, 1)
gemm_fused_pair_kernel(const __grid_constant__ CUtensorMap map_a, const FusedParams p) {
    constexpr int PER = codes_per_word(LV);
    constexpr int KPU = (PER == 16) ? 2 : 1;           // k-blocks covered by one packed slice (16 words per row)
    constexpr int ROWS = BN / 2;                       // channel rows this CTA expands
    constexpr int GROUPS = ROWS * 4;                   // 16-byte groups (four words of one row) per slice
    constexpr int TASKS = (GROUPS + 32 * kGroupWarps - 1) / (32 * kGroupWarps);
    constexpr uint32_t P_BYTES = ROWS * 64;            // one packed slice of this CTA's half tile
    static_assert(ROWS % 16 == 0, "half tiles are whole 16-row blocks");
    constexpr uint32_t A_BYTES = kGemmBM * kGemmBK, B_BYTES = ROWS * kGemmBK, STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TMEM_COLS = (2 * BN <= 256) ? 256 : 512;
    // D = s32, A = s8 (activations), B = u8 (codes), both K-major, N = BN, M = 256 across the pair
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (0u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                               (static_cast<uint32_t>(256 >> 4) << 24);

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* pring = smem + kFusedPairStages * STAGE;
    uint64_t* full = reinterpret_cast<uint64_t*>(pring + kPackedSlots * P_BYTES);
    uint64_t* empty = full + kFusedPairStages;
    uint64_t* pfull = empty + kFusedPairStages;
    uint64_t* pempty = pfull + kPackedSlots;
    uint64_t* tfull = pempty + kPackedSlots;
    uint64_t* tempty = tfull + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* fail = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = (rank == 0);
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int m_tiles = (p.M + 2 * kGemmBM - 1) / (2 * kGemmBM);
    const int n_tiles = (p.N + BN - 1) / BN;
    const int num_tiles = m_tiles * n_tiles;
    const int k_blocks = (p.K + kGemmBK - 1) / kGemmBK;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kFusedPairStages; ++s) {
            mbar_init(&full[s], 1 + 2 * kGroupWarps);  // leader's expect_tx + the expander warps (one group) of both CTAs
            mbar_init(&empty[s], 1);                            // tcgen05.commit (multicast to both CTAs)
        }
        for (int s = 0; s < kPackedSlots; ++s) {
            mbar_init(&pfull[s], 1);                      // this CTA's producer (expect_tx)
            mbar_init(&pempty[s], kGroupWarps);           // this CTA's expander warps (one group)
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull[b], 1);
            mbar_init(&tempty[b], 8);  // four epilogue warps of each CTA, all arriving at the leader
        }
        *fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything can signal them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        // activations by TMA, one tile per k-block; packed codes by bulk copy, one slice per KPU k-blocks.
        // The packed weights do not depend on the previous kernel, the activations do.
        if (lane == 0) {
            const int words_per_row = p.K / PER;
            const size_t rb_words = static_cast<size_t>(16) * round_up16(words_per_row);  // words per 16-row block
            const int rb_total = (p.N + 15) >> 4;
            bool waited = false;
            uint32_t it = 0, pit = 0;
            for (int tile = pair; tile < num_tiles && !*fail; tile += npairs) {
                const int m0 = (tile % m_tiles) * 2 * kGemmBM + static_cast<int>(rank) * kGemmBM;  // this CTA's tokens
                const int rb0 = ((tile / m_tiles) * BN + static_cast<int>(rank) * ROWS) >> 4;       // its first 16-row block
                const int rb_valid = max(0, min(ROWS / 16, rb_total - rb0));
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    if (kb % KPU == 0) {  // next packed slice
                        const int ps = pit % kPackedSlots;
                        if (pit >= kPackedSlots && !mbar_wait(&pempty[ps], ((pit / kPackedSlots) - 1) & 1, 45)) {
                            *fail = 1;
                            break;
                        }
                        const int sl = kb / KPU;  // slice index along K: tile sl / 8, slice sl % 8 inside it
                        mbar_expect_tx(&pfull[ps], static_cast<uint32_t>(rb_valid) * 1024u);
                        for (int rb = 0; rb < rb_valid; ++rb)
                            bulk_g2s(pring + ps * P_BYTES + rb * 1024,
                                     p.packed + (rb0 + rb) * rb_words + static_cast<size_t>(sl >> 3) * (kTileRows * kChunkWords) +
                                         (sl & 7) * 256,
                                     1024, &pfull[ps]);
                        ++pit;
                    }
                    if (!waited) {
                        pdl_wait();
                        waited = true;
                    }
                    const int s = it % kFusedPairStages;
                    if (it >= kFusedPairStages && !mbar_wait(&empty[s], ((it / kFusedPairStages) - 1) & 1, 40)) {
                        *fail = 1;
                        break;
                    }
                    if (leader) mbar_expect_tx(&full[s], 2 * A_BYTES);
                    tma_load_2d_pair(smem + s * STAGE, &map_a, kb * kGemmBK, m0, &full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        pdl_wait();
        if (leader && lane == 0) {
            uint32_t it = 0, tcount = 0;
            for (int tile = pair; tile < num_tiles && !*fail; tile += npairs, ++tcount) {
                const int buf = tcount & 1;
                if (tcount >= 2 && !mbar_wait(&tempty[buf], ((tcount >> 1) - 1) & 1, 41)) {
                    *fail = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kFusedPairStages;
                    if (!mbar_wait(&full[s], (it / kFusedPairStages) & 1, 42)) {
                        *fail = 1;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + s * STAGE);
                    const uint64_t adesc = make_kmajor_sw128_desc(a_addr);
                    const uint64_t bdesc = make_kmajor_sw128_desc(a_addr + A_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < kGemmBK / 32; ++k4)
                        tc_mma_i8_pair(d_addr, adesc + 2 * k4, bdesc + 2 * k4, IDESC, (kb | k4) != 0);
                    tc_commit_pair(&empty[s]);
                }
                if (*fail) break;
                tc_commit_pair(&tfull[buf]);
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue warps (both CTAs)
        pdl_wait();
        const int quarter = warp & 3;
        uint32_t tcount = 0;
        for (int tile = pair; tile < num_tiles; tile += npairs, ++tcount) {
            const int mt = tile % m_tiles, nt = tile / m_tiles;
            const int buf = tcount & 1;
            const int m = mt * 2 * kGemmBM + static_cast<int>(rank) * kGemmBM + quarter * 32 + lane;
            const float sa = (m < p.M) ? p.s_a[m] : 0.0f;
            const int sq = (m < p.M) ? p.sumq[m] : 0;
            if (!mbar_wait(&tfull[buf], (tcount >> 1) & 1, 43)) {
                *fail = 1;
                break;
            }
            tc_fence_after();
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN + c0, v);
                tc_wait_ld();
                const int nbase = nt * BN + c0;
                if (m < p.M && nbase < p.N) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = static_cast<uint32_t>(fused_level_sum<LV>(static_cast<int>(v[j]), sq));
                    const size_t o = static_cast<size_t>(m) * p.N + nbase;
                    const bool whole = (nbase + 32 <= p.N) && ((p.N & 7) == 0);
                    if (p.acc_debug) {
                        for (int j = 0; j < 32; ++j)
                            if (nbase + j < p.N) p.acc_debug[o + j] = static_cast<int>(v[j]);
                    }
                    if (whole) {
                        if (p.y_bf16) {
                            uint32_t h[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float y0 = scale_epilogue(static_cast<int>(v[2 * j]), sa, __ldg(p.s_n + nbase + 2 * j));
                                const float y1 = scale_epilogue(static_cast<int>(v[2 * j + 1]), sa, __ldg(p.s_n + nbase + 2 * j + 1));
                                h[j] = static_cast<uint32_t>(f32_to_bf16_bits(y0)) | (static_cast<uint32_t>(f32_to_bf16_bits(y1)) << 16);
                            }
                            uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(p.Y) + o);
#pragma unroll
                            for (int j = 0; j < 4; ++j) dst[j] = make_uint4(h[4 * j], h[4 * j + 1], h[4 * j + 2], h[4 * j + 3]);
                        } else {
                            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.Y) + o);
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float4 f;
                                f.x = scale_epilogue(static_cast<int>(v[4 * j]), sa, __ldg(p.s_n + nbase + 4 * j));
                                f.y = scale_epilogue(static_cast<int>(v[4 * j + 1]), sa, __ldg(p.s_n + nbase + 4 * j + 1));
                                f.z = scale_epilogue(static_cast<int>(v[4 * j + 2]), sa, __ldg(p.s_n + nbase + 4 * j + 2));
                                f.w = scale_epilogue(static_cast<int>(v[4 * j + 3]), sa, __ldg(p.s_n + nbase + 4 * j + 3));
                                dst[j] = f;
                            }
                        }
                    } else {
                        for (int j = 0; j < 32; ++j) {
                            if (nbase + j < p.N) {
                                const float y = scale_epilogue(static_cast<int>(v[j]), sa, p.s_n[nbase + j]);
                                if (p.y_bf16) static_cast<uint16_t*>(p.Y)[o + j] = f32_to_bf16_bits(y);
                                else static_cast<float*>(p.Y)[o + j] = y;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(&tempty[buf]);
        }
    } else {
        // ------------------------------------------------------------------ expander warps (both CTAs)
        // A thread's task is one 16-byte group of the slice: four words of one row.  Two-bit codes: that
        // is half of the row's 128-byte line in k-block (quad / 2) of the slice; INT4: a quarter of the
        // row's line in the slice's only k-block.  Groups are taken in storage order, so a warp reads
        // 512 contiguous bytes.
        const int et = (threadIdx.x - 6 * 32) % (32 * kGroupWarps);   // index inside the expander group
        const int egroup = (threadIdx.x - 6 * 32) / (32 * kGroupWarps);
        const uint32_t my_tiles = (pair < num_tiles) ? (num_tiles - pair + npairs - 1) / npairs : 0;
        const int rb_total = (p.N + 15) >> 4;
        const int slices_per_tile = (k_blocks + KPU - 1) / KPU;
        bool ok = true;
        for (uint32_t t = 0; t < my_tiles && ok; ++t) {
            const int tile = pair + static_cast<int>(t) * npairs;
            const int rb0 = ((tile / m_tiles) * BN + static_cast<int>(rank) * ROWS) >> 4;
            const int rb_valid = max(0, min(ROWS / 16, rb_total - rb0));
            for (int sl = 0; sl < slices_per_tile && ok; ++sl) {
                const uint32_t pit = t * slices_per_tile + sl;           // slice number in this CTA's sequence
                if (static_cast<int>(pit % kExpanderGroups) != egroup) continue;
                const uint32_t it = t * k_blocks + sl * KPU;             // k-block number of the slice's first k-block
                const int ps = pit % kPackedSlots;
                const int nkb = min(KPU, k_blocks - sl * KPU);           // k-blocks of this slice that exist
                if (!mbar_wait(&pfull[ps], (pit / kPackedSlots) & 1, 46)) ok = false;
                for (int j = 0; j < nkb && ok; ++j) {
                    const uint32_t i2 = it + j;
                    if (i2 >= kFusedPairStages && !mbar_wait(&empty[i2 % kFusedPairStages], ((i2 / kFusedPairStages) - 1) & 1, 44))
                        ok = false;
                }
                if (!ok) {
                    *fail = 1;
                    break;
                }
#pragma unroll
                for (int task = 0; task < TASKS; ++task) {
                    const int g = et + task * 32 * kGroupWarps;
                    if (g < GROUPS) {
                        const int rb = g >> 6, row = (rb << 4) + (((g >> 5) & 1) << 3) + ((g >> 2) & 7), quad = g & 3;
                        uint4 w4 = make_uint4(0, 0, 0, 0);
                        if (rb < rb_valid) w4 = *reinterpret_cast<const uint4*>(pring + ps * P_BYTES + g * 16);
                        const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
                        if constexpr (PER == 16) {
                            if ((quad >> 1) < nkb) {
                                unsigned char* bst = smem + ((it + (quad >> 1)) % kFusedPairStages) * STAGE + A_BYTES + row * 128;
#pragma unroll
                                for (int i = 0; i < 4; ++i)  // word i = 16 codes = one 16-byte chunk
                                    *reinterpret_cast<uint4*>(bst + ((((quad & 1) << 2) + i) ^ (row & 7)) * 16) =
                                        make_uint4(operand_word<LV>(w[i], 0), operand_word<LV>(w[i], 1), operand_word<LV>(w[i], 2),
                                                   operand_word<LV>(w[i], 3));
                            }
                        } else {
                            unsigned char* bst = smem + (it % kFusedPairStages) * STAGE + A_BYTES + row * 128;
#pragma unroll
                            for (int i = 0; i < 2; ++i)  // two words (8 codes each) make one 16-byte chunk
                                *reinterpret_cast<uint4*>(bst + (((quad << 1) + i) ^ (row & 7)) * 16) =
                                    make_uint4(operand_word<LV>(w[2 * i], 0), operand_word<LV>(w[2 * i], 1),
                                               operand_word<LV>(w[2 * i + 1], 0), operand_word<LV>(w[2 * i + 1], 1));
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> tensor core
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&pempty[ps]);
                    for (int j = 0; j < nkb; ++j) mbar_arrive_leader(&full[(it + j) % kFusedPairStages]);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while the other may still use it
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace qift

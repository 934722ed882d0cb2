// Prefill GEMM on CTA pairs (cta_group::2): two SMs share one 256-token x BN-channel output tile.
//
// With one CTA per tile (gemm_i8_tcgen05_kernel) every 128-byte k-block needs 16 KB of activations
// and 32 KB of weights in shared memory for 128x256x128 MACs; at the int8 rate of the tensor core
// that is 92 B/clk/SM, and with ~190 KB of stages in flight against ~2 us of L2 latency the pipe
// idles almost half of the time.  A CTA pair halves the weight traffic: each CTA loads its own 128
// tokens and only HALF of the tile's channels; tcgen05.mma.cta_group::2 (issued by the leader CTA)
// reads the weight halves of both CTAs and writes 128 accumulator rows into each CTA's tensor memory.
// Per k-block a CTA now stages 16 + 16 KB for the same MACs, in a 6-deep ring.
//
// Protocol (no TMA multicast anywhere):
//   * both CTAs' producers load with cp.async.bulk.tensor...cta_group::2, whose completion bytes are
//     counted on the LEADER's full barrier (barrier address with the CTA-rank bit cleared); only the
//     leader's producer arms it (expect_tx of both CTAs' bytes);
//   * the leader's MMA thread frees a ring slot / publishes an accumulator with tcgen05.commit
//     multicast to the same barrier in both CTAs;
//   * both CTAs' epilogue warps release an accumulator buffer by arriving on the leader's barrier
//     (the peer through its shared::cluster address);
//   * cluster barriers after set-up and before tear-down keep either CTA from touching the other's
//     shared memory or barriers outside its lifetime.
// Every wait is bounded; on expiry the kernel records the site, stops and still frees tensor memory.
//
// One launch may serve several products that share the activations (q/k/v; gate/up): the channel
// tiles of all of them form one list ("segments": each with its own decoded weights, channel
// scales and output), so that a narrow product does not leave most SM pairs idle for a round.
//
// Side job: the GEMM leaves most issue slots of an SM unused, and the decoding of packed codes
// into the int8 levels that the NEXT product will read needs nothing this product computes.  Eight
// extra warps per CTA therefore run a list of such decoding jobs (units of 8 channels x 128
// packed words) beside the GEMM; they touch neither the pipeline's barriers nor its shared memory.
#pragma once

#include "common.cuh"
#include "prefill.cuh"

namespace qift {

constexpr int kPairGemmThreads = 192;                      // producer, MMA issuer, four epilogue warps
constexpr int kPairSideWarps = 8;                          // warps that decode the NEXT product's codes meanwhile
constexpr int kPairThreads = kPairGemmThreads + 32 * kPairSideWarps;
constexpr int kPairStages = 6;
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;  // clears the CTA-rank bit of a shared::cluster address (rank 1 -> rank 0)

__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
            smem_u32(dst)),
        "l"(map), "r"(smem_u32(bar) & kPeerBitMask), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive (once the preceding MMAs have completed) on the barrier at this shared-memory offset in both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                     smem_u32(bar)),
                 "h"(static_cast<uint16_t>(3))
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(uint64_t* bar) {  // same offset, CTA rank 0 of the pair
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(smem_u32(bar) & kPeerBitMask) : "memory");
}

template <int BN>
__host__ __device__ constexpr size_t pair_smem_bytes() {
    return 1024 + static_cast<size_t>(kPairStages) * (kGemmBM * kGemmBK + (BN / 2) * kGemmBK) + 256;
}

constexpr int kPairMaxSegments = 4;
constexpr int kPairMaxJobs = 8;   // matrices decoded on the side in one launch (they may belong to several later calls)
constexpr int kSideUnitRows = 8, kSideUnitWords = 128;

struct PairSegment {
    const float* s_n;    // [N]
    void* Y;             // [M, N]
    int32_t* acc_debug;  // [M, N] or null
    int N;
    int tile0;           // index of the segment's first channel tile in the launch's list
};
struct SideJob {         // decode packed[N rows, words_per_row] -> int8 out[N, K]
    const uint32_t* packed;
    int8_t* out;
    int N, words_per_row;
    int unit0;           // index of the job's first unit in the launch's list
    int levels;
};
struct alignas(64) PairParams {
    CUtensorMap map_a;                    // q_a [M, K]
    CUtensorMap map_b[kPairMaxSegments];  // decoded weights [N_i, K], box = BN / 2 rows
    PairSegment seg[kPairMaxSegments];
    SideJob job[kPairMaxJobs];
    const float* s_a;
    uint64_t wait_limit_ns;  // bound of every device-side wait of the launch; 0 = the default (kWaitLimitNs)
    int M, K, y_bf16;
    int nseg, n_tiles;       // segments, channel tiles over all of them
    int njobs, units;        // side jobs, units over all of them
    int starve;              // self-test only (qift_selftest_wait_timeout): the producers issue no loads
};

// Side-job units: eight channel rows x 128 packed words, a word of each row per thread of a 128-thread group.
// A thread works on two units at a time: sixteen loads in flight, then sixteen 16-byte stores (a warp writes
// 512 contiguous bytes of a row per store instruction).
struct SideUnit {
    const uint32_t* src;  // the thread's word of the unit's first row (rows are 16 words apart in the tiled layout)
    int8_t* dst;          // its 16 (INT4: 8) level bytes of the first row
    int rows;             // rows of the unit that exist (0 = nothing to do)
    size_t row_bytes;     // K
};
__device__ __forceinline__ SideUnit side_unit(const SideJob& j, int unit, int t) {
    const int per = codes_per_word(j.levels);
    const int chunks = (j.words_per_row + kSideUnitWords - 1) / kSideUnitWords;
    const int rb = unit / chunks;
    const int n0 = rb * kSideUnitRows, jw = (unit - rb * chunks) * kSideUnitWords + t;
    SideUnit u;
    u.rows = (jw < j.words_per_row) ? min(kSideUnitRows, j.N - n0) : 0;
    u.src = j.packed + packed_word_address(n0, jw, round_up16(j.words_per_row));
    u.row_bytes = static_cast<size_t>(j.words_per_row) * per;
    u.dst = j.out + static_cast<size_t>(n0) * u.row_bytes + static_cast<size_t>(jw) * per;
    return u;
}
template <int LV>
__device__ __forceinline__ void side_store(const SideUnit& u, const uint32_t (&w)[kSideUnitRows]) {
    constexpr int PER = codes_per_word(LV);
#pragma unroll
    for (int r = 0; r < kSideUnitRows; ++r) {
        if (r >= u.rows) break;
        uint32_t v[PER / 4];
        expand_word<LV>(w[r], v);
        int8_t* d = u.dst + r * u.row_bytes;
        if constexpr (PER == 16) *reinterpret_cast<uint4*>(d) = make_uint4(v[0], v[1], v[2], v[3]);
        else *reinterpret_cast<uint2*>(d) = make_uint2(v[0], v[1]);
    }
}
__device__ __forceinline__ void side_store_any(int levels, const SideUnit& u, const uint32_t (&w)[kSideUnitRows]) {
    switch (levels) {
        case QIFT_LEVELS_MNZ: side_store<QIFT_LEVELS_MNZ>(u, w); break;
        case QIFT_LEVELS_POT: side_store<QIFT_LEVELS_POT>(u, w); break;
        case QIFT_LEVELS_SYM: side_store<QIFT_LEVELS_SYM>(u, w); break;
        default: side_store<QIFT_LEVELS_INT4>(u, w); break;
    }
}

// The side warps' loop: groups of 128 threads; group q of CTA b takes units 2 (b * groups + q), + 1, then strides on.
__device__ __forceinline__ void side_jobs(const PairParams& p, int t, int group) {
    constexpr int kGroups = 32 * kPairSideWarps / kSideUnitWords;
    auto job_of = [&](int u) {
        int ji = 0;
#pragma unroll
        for (int i = 1; i < kPairMaxJobs; ++i)
            if (i < p.njobs && u >= p.job[i].unit0) ji = i;
        return ji;
    };
    for (int u0 = 2 * (blockIdx.x * kGroups + group); u0 < p.units; u0 += 2 * gridDim.x * kGroups) {
        const int ja = job_of(u0), jb = job_of(min(u0 + 1, p.units - 1));
        SideUnit a = side_unit(p.job[ja], u0 - p.job[ja].unit0, t);
        SideUnit b = side_unit(p.job[jb], u0 + 1 - p.job[jb].unit0, t);
        if (u0 + 1 >= p.units) b.rows = 0;
        uint32_t wa[kSideUnitRows], wb[kSideUnitRows];
#pragma unroll
        for (int r = 0; r < kSideUnitRows; ++r) wa[r] = (r < a.rows) ? __ldg(a.src + 16 * r) : 0u;
#pragma unroll
        for (int r = 0; r < kSideUnitRows; ++r) wb[r] = (r < b.rows) ? __ldg(b.src + 16 * r) : 0u;
        side_store_any(p.job[ja].levels, a, wa);
        side_store_any(p.job[jb].levels, b, wb);
    }
}

template <int BN>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_i8_pair_kernel(const __grid_constant__ PairParams p) {
    constexpr uint32_t A_BYTES = kGemmBM * kGemmBK, B_BYTES = (BN / 2) * kGemmBK, STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TMEM_COLS = (2 * BN <= 256) ? 256 : 512;
    // D = s32, A = B = s8, both K-major, N = BN, M = 256 across the pair
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                               (static_cast<uint32_t>(256 >> 4) << 24);

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kPairStages * STAGE);
    uint64_t* empty = full + kPairStages;
    uint64_t* tfull = empty + kPairStages;
    uint64_t* tempty = tfull + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* fail = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = (rank == 0);
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int m_tiles = (p.M + 2 * kGemmBM - 1) / (2 * kGemmBM);
    const int num_tiles = m_tiles * p.n_tiles;
    const int k_blocks = (p.K + kGemmBK - 1) / kGemmBK;
    const uint64_t limit = p.wait_limit_ns ? p.wait_limit_ns : kWaitLimitNs;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(&full[s], 1);   // armed by the leader's producer; bytes arrive from both CTAs
            mbar_init(&empty[s], 1);  // tcgen05.commit (multicast to both CTAs)
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull[b], 1);   // tcgen05.commit (multicast)
            mbar_init(&tempty[b], 8);  // four epilogue warps of each CTA, all arriving at the leader
        }
        *fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&p.map_a);
        for (int s = 0; s < p.nseg; ++s) tma_prefetch_desc(&p.map_b[s]);
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
    pdl_wait();

    // channel tile g of the launch's list -> its segment
    auto segment_of = [&](int g) {
        int s = 0;
#pragma unroll
        for (int i = 1; i < kPairMaxSegments; ++i)
            if (i < p.nseg && g >= p.seg[i].tile0) s = i;
        return s;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0 && !p.starve) {
            uint32_t it = 0;
            for (int tile = pair; tile < num_tiles && !*fail; tile += npairs) {
                const int mt = tile % m_tiles, g = tile / m_tiles;
                const int sg = segment_of(g);
                const int m0 = mt * 2 * kGemmBM + static_cast<int>(rank) * kGemmBM;           // this CTA's tokens
                const int n0 = (g - p.seg[sg].tile0) * BN + static_cast<int>(rank) * (BN / 2);  // this CTA's half of the channels
                const CUtensorMap* mb = &p.map_b[sg];
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (it >= kPairStages && !mbar_wait(&empty[s], ((it / kPairStages) - 1) & 1, 30, limit)) {
                        *fail = 1;
                        break;
                    }
                    if (leader) mbar_expect_tx(&full[s], 2 * STAGE);
                    tma_load_2d_pair(smem + s * STAGE, &p.map_a, kb * kGemmBK, m0, &full[s]);
                    tma_load_2d_pair(smem + s * STAGE + A_BYTES, mb, kb * kGemmBK, n0, &full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (leader && lane == 0) {
            uint32_t it = 0, tcount = 0;
            for (int tile = pair; tile < num_tiles && !*fail; tile += npairs, ++tcount) {
                const int buf = tcount & 1;
                if (tcount >= 2 && !mbar_wait(&tempty[buf], ((tcount >> 1) - 1) & 1, 31, limit)) {
                    *fail = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (!mbar_wait(&full[s], (it / kPairStages) & 1, 32, limit)) {
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
        const int quarter = warp & 3;
        uint32_t tcount = 0;
        for (int tile = pair; tile < num_tiles; tile += npairs, ++tcount) {
            const int mt = tile % m_tiles, g = tile / m_tiles;
            const int sg = segment_of(g);
            const PairSegment& S = p.seg[sg];
            const int N = S.N;
            const int buf = tcount & 1;
            if (!mbar_wait(&tfull[buf], (tcount >> 1) & 1, 33, limit)) {
                *fail = 1;
                break;
            }
            tc_fence_after();
            const int m = mt * 2 * kGemmBM + static_cast<int>(rank) * kGemmBM + quarter * 32 + lane;
            const float sa = (m < p.M) ? p.s_a[m] : 0.0f;
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN + c0, v);
                tc_wait_ld();
                const int nbase = (g - S.tile0) * BN + c0;
                if (m < p.M && nbase < N) {
                    const size_t o = static_cast<size_t>(m) * N + nbase;
                    const bool whole = (nbase + 32 <= N) && ((N & 7) == 0);
                    if (S.acc_debug) {
                        for (int j = 0; j < 32; ++j)
                            if (nbase + j < N) S.acc_debug[o + j] = static_cast<int>(v[j]);
                    }
                    if (whole) {
                        if (p.y_bf16) {
                            uint32_t h[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float y0 = scale_epilogue(static_cast<int>(v[2 * j]), sa, __ldg(S.s_n + nbase + 2 * j));
                                const float y1 = scale_epilogue(static_cast<int>(v[2 * j + 1]), sa, __ldg(S.s_n + nbase + 2 * j + 1));
                                h[j] = static_cast<uint32_t>(f32_to_bf16_bits(y0)) | (static_cast<uint32_t>(f32_to_bf16_bits(y1)) << 16);
                            }
                            uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(S.Y) + o);
#pragma unroll
                            for (int j = 0; j < 4; ++j) dst[j] = make_uint4(h[4 * j], h[4 * j + 1], h[4 * j + 2], h[4 * j + 3]);
                        } else {
                            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(S.Y) + o);
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float4 f;
                                f.x = scale_epilogue(static_cast<int>(v[4 * j]), sa, __ldg(S.s_n + nbase + 4 * j));
                                f.y = scale_epilogue(static_cast<int>(v[4 * j + 1]), sa, __ldg(S.s_n + nbase + 4 * j + 1));
                                f.z = scale_epilogue(static_cast<int>(v[4 * j + 2]), sa, __ldg(S.s_n + nbase + 4 * j + 2));
                                f.w = scale_epilogue(static_cast<int>(v[4 * j + 3]), sa, __ldg(S.s_n + nbase + 4 * j + 3));
                                dst[j] = f;
                            }
                        }
                    } else {
                        for (int j = 0; j < 32; ++j) {
                            if (nbase + j < N) {
                                const float y = scale_epilogue(static_cast<int>(v[j]), sa, S.s_n[nbase + j]);
                                if (p.y_bf16) static_cast<uint16_t*>(S.Y)[o + j] = f32_to_bf16_bits(y);
                                else static_cast<float*>(S.Y)[o + j] = y;
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
        // ------------------------------------------------------------------ side warps: decode the next product's codes
        const int t = (threadIdx.x - kPairGemmThreads) & (kSideUnitWords - 1);
        const int group = (threadIdx.x - kPairGemmThreads) / kSideUnitWords;
        side_jobs(p, t, group);
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

// Prefill-path product (M > 16): the packed codes are expanded once per call to an int8 [N,K]
// scratch (the decoded levels), then a persistent TMA-fed tcgen05 kind::i8 GEMM with INT32
// accumulators in tensor memory computes acc[m,n] = sum_k q_a[m,k] * level[n,k] and applies the
// scales in its epilogue.
//
// GEMM structure (one CTA per SM, 192 threads):
//   warp 0      TMA producer: per 128-byte k-block one box of A (128 tokens x 128 B) and one box of
//               B (BN channels x 128 B), 128-byte swizzle, into a 4-deep shared-memory ring
//   warp 1      allocates tensor memory, issues tcgen05.mma (M=128, N=BN, K=32 per instruction),
//               frees ring slots and publishes finished accumulators through tcgen05.commit
//   warps 2-5   epilogue: tcgen05.ld the accumulator (lane = token, column = channel), scale, store
// Two accumulator buffers in tensor memory let the epilogue of tile i overlap the mainloop of i+1.
// Every wait is bounded; on expiry the kernel records the site, skips its work and still frees
// tensor memory.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace qift {

// ------------------------------------------------------------------------------------------------
// expansion: packed codes -> int8 levels, K contiguous
// ------------------------------------------------------------------------------------------------
// One packed word -> its PER level bytes in k order (o[t] holds codes 4t .. 4t+3).  Four codes (one per byte of
// w, at bit (32 / PER) * t of the byte) become four level bytes at once: the low bits of a level are the code's
// bits with one of them flipped; the sign extension is all ones exactly when one bit of that intermediate is
// set, and comes from a multiply that cannot carry across bytes.
template <int LV>
__device__ __forceinline__ void expand_word(uint32_t w, uint32_t (&o)[codes_per_word(LV) / 4]) {
    constexpr int PER = codes_per_word(LV);
#pragma unroll
    for (int t = 0; t < PER / 4; ++t) {
        if constexpr (LV == QIFT_LEVELS_MNZ) {         // 2c - 3: low three bits (2c) ^ 5, bits 3..7 set iff c < 2
            const uint32_t x = (t == 0) ? (w << 1) : (w >> (2 * t - 1));
            const uint32_t u = (x & 0x06060606u) ^ 0x05050505u;
            o[t] = (u & 0x04040404u) * 62u + u;
        } else if constexpr (LV == QIFT_LEVELS_SYM) {  // c - 2: low two bits c ^ 2, bits 2..7 set iff c < 2
            const uint32_t u = ((w >> (2 * t)) & 0x03030303u) ^ 0x02020202u;
            o[t] = (u & 0x02020202u) * 126u + u;
        } else if constexpr (LV == QIFT_LEVELS_INT4) { // nibble sign-extended: bits 4..7 set iff bit 3
            const uint32_t u = (w >> (4 * t)) & 0x0f0f0f0fu;
            o[t] = (u & 0x08080808u) * 30u + u;
        } else {                                       // PoT: code by code
            uint32_t r = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int code = (w >> (8 * b + (32 / PER) * t)) & ((1u << (32 / PER)) - 1u);
                r |= (static_cast<uint32_t>(level_from_code<LV>(code)) & 0xffu) << (8 * b);
            }
            o[t] = r;
        }
    }
}

// Blocks of eight rows are dealt to the CTAs, the words of a row to the threads (no division per word).  A thread
// asks for its word of all eight rows before it uses the first (with one 4-byte load per thread in flight the
// kernel was bound by the latency of that load: 0.9 TB/s read, ncu's long-scoreboard stall 12 cycles per issue;
// the eight rows of a block also make one contiguous 512-byte piece of the packed layout per 16-word slice) and
// writes the 16 (W4: 8) level bytes of each word with one store.  (Four words per thread, one 128-bit load and 64 bytes written,
// was measured slower: a row of 4096 weights then occupies a quarter of the CTA.)
constexpr int kExpandRows = 8;

template <int LV>
__global__ void __launch_bounds__(256)
expand_levels_kernel(const uint32_t* __restrict__ packed, int N, int words_per_row, int8_t* __restrict__ out) {
    constexpr int PER = codes_per_word(LV);
    pdl_launch_dependents();
    pdl_wait();
    const int pitch = round_up16(words_per_row);
    for (int n0 = blockIdx.x * kExpandRows; n0 < N; n0 += gridDim.x * kExpandRows)
        for (int jw = threadIdx.x; jw < words_per_row; jw += blockDim.x) {
            uint32_t w[kExpandRows], wh[kExpandRows];
#pragma unroll
            for (int r = 0; r < kExpandRows; ++r) {
                if constexpr (LV == QIFT_LEVELS_INT3) {   // the low word and the high word it shares with its neighbour
                    w[r] = (n0 + r < N) ? packed[int3_low_address(n0 + r, jw, pitch)] : 0u;
                    wh[r] = (n0 + r < N) ? packed[int3_high_address(n0 + r, jw, pitch)] : 0u;
                } else {
                    w[r] = (n0 + r < N) ? packed[packed_word_address(n0 + r, jw, pitch)] : 0u;
                    wh[r] = 0u;
                }
            }
#pragma unroll
            for (int r = 0; r < kExpandRows; ++r) {
                if (n0 + r >= N) break;
                const size_t j = static_cast<size_t>(n0 + r) * words_per_row + jw;
                uint32_t o[PER / 4];
                if constexpr (LV == QIFT_LEVELS_INT3) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) o[t] = int3_level_bytes(w[r], wh[r], jw, t);
                } else {
                    expand_word<LV>(w[r], o);
                }
                if constexpr (PER == 16) reinterpret_cast<uint4*>(out)[j] = make_uint4(o[0], o[1], o[2], o[3]);
                else reinterpret_cast<uint2*>(out)[j] = make_uint2(o[0], o[1]);
            }
        }
}

// ------------------------------------------------------------------------------------------------
// tcgen05 / TMA wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
            smem_u32(dst)),
        "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_mma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand tile with 128-byte swizzle: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);  // start address
    d |= static_cast<uint64_t>(1) << 16;                      // leading byte offset (unused with swizzle)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;              // stride byte offset between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                      // descriptor version (sm_100)
    d |= static_cast<uint64_t>(2) << 61;                      // SWIZZLE_128B
    return d;
}

constexpr int kGemmThreads = 192;
constexpr int kGemmBM = 128;
constexpr int kGemmBK = 128;  // bytes = int8 elements per k-block
constexpr int kGemmStages = 4;

struct GemmParams {
    const float* s_n;
    const float* s_a;
    void* Y;
    int32_t* acc_debug;
    int M, N, K;
    int y_bf16;
};

template <int BN>
__host__ __device__ constexpr size_t gemm_smem_bytes() {
    return 1024 /*alignment slack*/ + static_cast<size_t>(kGemmStages) * (kGemmBM * kGemmBK + BN * kGemmBK) + 256;
}

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_i8_tcgen05_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const GemmParams p) {
    constexpr uint32_t A_BYTES = kGemmBM * kGemmBK, B_BYTES = BN * kGemmBK, STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TMEM_COLS = (2 * BN <= 32) ? 32 : (2 * BN <= 64) ? 64 : (2 * BN <= 128) ? 128 : (2 * BN <= 256) ? 256 : 512;
    // instruction descriptor: D = s32, A = B = s8, both K-major, N = BN, M = 128
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                               (static_cast<uint32_t>(kGemmBM >> 4) << 24);

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kGemmStages * STAGE);
    uint64_t* empty = full + kGemmStages;
    uint64_t* tfull = empty + kGemmStages;
    uint64_t* tempty = tfull + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* fail = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m_tiles = (p.M + kGemmBM - 1) / kGemmBM;
    const int n_tiles = (p.N + BN - 1) / BN;
    const int num_tiles = m_tiles * n_tiles;
    const int k_blocks = (p.K + kGemmBK - 1) / kGemmBK;

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemmStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull[b], 1);
            mbar_init(&tempty[b], 4);
        }
        *fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !*fail; tile += gridDim.x) {
                const int mt = tile % m_tiles, nt = tile / m_tiles;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kGemmStages;
                    if (it >= kGemmStages && !mbar_wait(&empty[s], ((it / kGemmStages) - 1) & 1, 10)) {
                        *fail = 1;
                        break;
                    }
                    mbar_expect_tx(&full[s], STAGE);
                    tma_load_2d(smem + s * STAGE, &map_a, kb * kGemmBK, mt * kGemmBM, &full[s]);
                    tma_load_2d(smem + s * STAGE + A_BYTES, &map_b, kb * kGemmBK, nt * BN, &full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !*fail; tile += gridDim.x, ++tcount) {
                const int buf = tcount & 1;
                if (tcount >= 2 && !mbar_wait(&tempty[buf], ((tcount >> 1) - 1) & 1, 11)) {
                    *fail = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kGemmStages;
                    if (!mbar_wait(&full[s], (it / kGemmStages) & 1, 12)) {
                        *fail = 1;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + s * STAGE);
                    const uint64_t adesc = make_kmajor_sw128_desc(a_addr);
                    const uint64_t bdesc = make_kmajor_sw128_desc(a_addr + A_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < kGemmBK / 32; ++k4)  // 32 bytes of K per instruction: +2 in 16-byte units
                        tc_mma_i8(d_addr, adesc + 2 * k4, bdesc + 2 * k4, IDESC, (kb | k4) != 0);
                    tc_commit(&empty[s]);  // slot reusable once these MMAs have read it
                }
                if (*fail) break;
                tc_commit(&tfull[buf]);  // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;  // tensor-memory lane quarter this warp may read
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++tcount) {
            const int mt = tile % m_tiles, nt = tile / m_tiles;
            const int buf = tcount & 1;
            if (!mbar_wait(&tfull[buf], (tcount >> 1) & 1, 13)) {
                *fail = 1;
                break;
            }
            tc_fence_after();
            const int m = mt * kGemmBM + quarter * 32 + lane;
            const float sa = (m < p.M) ? p.s_a[m] : 0.0f;
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN + c0, v);
                tc_wait_ld();
                const int nbase = nt * BN + c0;
                if (m < p.M && nbase < p.N) {
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
            if (lane == 0) mbar_arrive(&tempty[buf]);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace qift

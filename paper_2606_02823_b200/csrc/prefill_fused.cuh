// Prefill-path product with the code expansion fused into the GEMM (M > 16, no N*K scratch).
//
// Same persistent tcgen05 kind::i8 pipeline as gemm_i8_tcgen05_kernel, but the weight operand never
// exists in global memory as int8: four "expander" warps read the packed codes (2 bits per weight,
// L2-resident after the first token tile touches them) straight into registers, turn every packed
// word into unsigned-byte operand words with one shift + one mask per four codes, and store them
// into the 128-byte-swizzled shared-memory stage the tensor core reads.  The tensor core multiplies
// UNSIGNED codes (b_format = u8) by the signed activations; the affine level map is undone in the
// epilogue with the per-token sum of q_a:  acc = alpha * sum code*q + gamma * sum q.
//
//   warp 0      TMA producer for the activation tile (128 tokens x 128 B per k-block)
//   warp 1      tensor-memory allocation + tcgen05.mma issue
//   warps 2-5   epilogue (tcgen05.ld, level map, scales, stores)
//   warps 6-13  expanders: ld.global packed words (4 k-blocks ahead, in registers) -> st.shared
// Per k-block the CTA now pulls 16 KB (activations) + 8 KB (packed weights) instead of 48 KB, and
// the separate expansion pass with its N*K bytes of scratch traffic is gone.
#pragma once

#include "common.cuh"
#include "prefill.cuh"

namespace qift {

constexpr int kFusedExpanderWarps = 8;
constexpr int kFusedThreads = 192 + 32 * kFusedExpanderWarps;  // 448
constexpr int kFusedDepth = 4;  // k-blocks of packed words held in registers per expander thread

struct FusedParams {
    const uint32_t* packed;
    const float* s_n;
    const float* s_a;
    const int* sumq;  // [M] sum_k q_a[m,k]
    void* Y;
    int32_t* acc_debug;
    int M, N, K;
    int y_bf16;
};

// sum_k q_a[m,k] for every token row: one warp per row.
__global__ void __launch_bounds__(256)
rowsum_q_kernel(const int8_t* __restrict__ q_a, int M, int K, int* __restrict__ sumq) {
    pdl_launch_dependents();
    pdl_wait();
    const int m = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (m >= M) return;
    const uint4* row = reinterpret_cast<const uint4*>(q_a + static_cast<size_t>(m) * K);
    int s = 0;
    for (int i = lane; i < K / 16; i += 32) {
        const uint4 v = row[i];
        s = dp4a_us(0x01010101u, v.x, s), s = dp4a_us(0x01010101u, v.y, s);
        s = dp4a_us(0x01010101u, v.z, s), s = dp4a_us(0x01010101u, v.w, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) sumq[m] = s;
}

// Four consecutive-k codes of plane t of a packed word, as the unsigned byte operand.
template <int LV>
__device__ __forceinline__ uint32_t operand_word(uint32_t w, int t) {
    if constexpr (LV == QIFT_LEVELS_INT4) {
        return ((w >> (4 * t)) & 0x0f0f0f0fu) ^ 0x08080808u;  // nibble ^ 8 = level + 8
    } else if constexpr (LV == QIFT_LEVELS_POT) {
        const uint32_t c = (w >> (2 * t)) & 0x03030303u;
        return c * 3u - ((c >> 1) & 0x01010101u);              // 0,3,5,8 = level + 4
    } else {
        return (w >> (2 * t)) & 0x03030303u;                   // the code itself
    }
}

template <int LV>
__device__ __forceinline__ int fused_level_sum(int v, int sq) {
    if constexpr (LV == QIFT_LEVELS_MNZ) return 2 * v - 3 * sq;
    if constexpr (LV == QIFT_LEVELS_SYM) return v - 2 * sq;
    if constexpr (LV == QIFT_LEVELS_POT) return v - 4 * sq;
    return v - 8 * sq;
}

template <int BN>
__host__ __device__ constexpr size_t fused_smem_bytes() {
    return 1024 + static_cast<size_t>(kGemmStages) * (kGemmBM * kGemmBK + BN * kGemmBK) + 256;
}

template <int LV, int BN>
__global__ void __launch_bounds__(kFusedThreads, 1)
gemm_fused_kernel(const __grid_constant__ CUtensorMap map_a, const FusedParams p) {
    constexpr int PER = codes_per_word(LV);
    constexpr int WPK = kGemmBK / PER;         // packed words per row per k-block (8 or 16)
    constexpr int QPK = WPK / 4;               // 16-byte loads per row per k-block (2 or 4)
    constexpr int TPR = (32 * kFusedExpanderWarps) / BN;  // expander threads per channel row (1 or 2)
    constexpr int QPT = QPK / TPR;             // 16-byte loads per expander thread per k-block
    constexpr uint32_t A_BYTES = kGemmBM * kGemmBK, B_BYTES = BN * kGemmBK, STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TMEM_COLS = (2 * BN <= 256) ? 256 : 512;
    // D = s32, A = s8 (activations), B = u8 (codes), both K-major, N = BN, M = 128
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (0u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
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
            mbar_init(&full[s], 1 + kFusedExpanderWarps);  // the activation TMA (expect_tx) + one arrival per expander warp
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull[b], 1);
            mbar_init(&tempty[b], 4);
        }
        *fail = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
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

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (activations)
        pdl_wait();
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !*fail; tile += gridDim.x) {
                const int mt = tile % m_tiles;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kGemmStages;
                    if (it >= kGemmStages && !mbar_wait(&empty[s], ((it / kGemmStages) - 1) & 1, 20)) {
                        *fail = 1;
                        break;
                    }
                    mbar_expect_tx(&full[s], A_BYTES);
                    tma_load_2d(smem + s * STAGE, &map_a, kb * kGemmBK, mt * kGemmBM, &full[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        pdl_wait();
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !*fail; tile += gridDim.x, ++tcount) {
                const int buf = tcount & 1;
                if (tcount >= 2 && !mbar_wait(&tempty[buf], ((tcount >> 1) - 1) & 1, 21)) {
                    *fail = 1;
                    break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + buf * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % kGemmStages;
                    if (!mbar_wait(&full[s], (it / kGemmStages) & 1, 22)) {
                        *fail = 1;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + s * STAGE);
                    const uint64_t adesc = make_kmajor_sw128_desc(a_addr);
                    const uint64_t bdesc = make_kmajor_sw128_desc(a_addr + A_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < kGemmBK / 32; ++k4)
                        tc_mma_i8(d_addr, adesc + 2 * k4, bdesc + 2 * k4, IDESC, (kb | k4) != 0);
                    tc_commit(&empty[s]);
                }
                if (*fail) break;
                tc_commit(&tfull[buf]);
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue warps
        pdl_wait();
        const int quarter = warp & 3;
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++tcount) {
            const int mt = tile % m_tiles, nt = tile / m_tiles;
            const int buf = tcount & 1;
            const int m = mt * kGemmBM + quarter * 32 + lane;
            const float sa = (m < p.M) ? p.s_a[m] : 0.0f;
            const int sq = (m < p.M) ? p.sumq[m] : 0;
            if (!mbar_wait(&tfull[buf], (tcount >> 1) & 1, 23)) {
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
            if (lane == 0) mbar_arrive(&tempty[buf]);
        }
    } else {
        // ------------------------------------------------------------------ expander warps
        // (the packed weights never depend on the previous kernel: no wait before reading them)
        const int et = threadIdx.x - 6 * 32;       // 0 .. 255
        const int row = et % BN;                    // channel row of the tile this thread expands
        const int q0 = (et / BN) * QPT;             // its first 16-byte group of the row's k-block
        const int words_per_row = p.K / PER;
        const int pitch = round_up16(words_per_row);
        const uint32_t my_tiles = (blockIdx.x < num_tiles) ? (num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
        const uint32_t total = my_tiles * k_blocks;
        // byte offsets of this thread's 16-byte chunks inside a stage's weight tile (128-byte swizzle)
        constexpr int CPT = (PER == 16) ? 4 * QPT : 2 * QPT;  // chunks per thread per k-block
        uint32_t chunk_off[CPT];
#pragma unroll
        for (int c = 0; c < CPT; ++c) chunk_off[c] = row * 128 + ((((PER == 16) ? 4 * q0 : 2 * q0) + c) ^ (row & 7)) * 16;

        uint4 ring[kFusedDepth][QPT];
        int l_tile = blockIdx.x, l_kb = 0;
        const uint32_t* l_row = nullptr;
        auto set_row = [&](int tile) {
            const int n = (tile / m_tiles) * BN + row;
            l_row = (n < p.N) ? p.packed + static_cast<size_t>(n >> 4) * 16 * pitch + ((n >> 3) & 1) * 128 + (n & 7) * 16 : nullptr;
        };
        auto load = [&](uint4 (&dst)[QPT]) {
            // word j0 = l_kb * WPK of the row: tile j0/128, slice, quad (see packed_word_address)
            const int j0 = l_kb * WPK;
            const size_t off = static_cast<size_t>(j0 >> 7) * (kTileRows * kChunkWords) + ((j0 & 127) >> 4) * 256 + ((j0 >> 2) & 3) * 4;
#pragma unroll
            for (int q = 0; q < QPT; ++q) {
                const bool ok = l_row != nullptr && (j0 + 4 * (q0 + q)) < words_per_row;
                dst[q] = ok ? __ldg(reinterpret_cast<const uint4*>(l_row + off) + q0 + q) : make_uint4(0, 0, 0, 0);
            }
            if (++l_kb == k_blocks) {
                l_kb = 0;
                l_tile += gridDim.x;
                if (l_tile < num_tiles) set_row(l_tile);
            }
        };
        auto store = [&](const uint4 (&src)[QPT], unsigned char* bst) {
#pragma unroll
            for (int q = 0; q < QPT; ++q) {
                const uint32_t w[4] = {src[q].x, src[q].y, src[q].z, src[q].w};
                if constexpr (PER == 16) {
                    // word i of this group = 16 codes = one 16-byte chunk
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        *reinterpret_cast<uint4*>(bst + chunk_off[4 * q + i]) =
                            make_uint4(operand_word<LV>(w[i], 0), operand_word<LV>(w[i], 1), operand_word<LV>(w[i], 2),
                                       operand_word<LV>(w[i], 3));
                } else {
                    // INT4: two words (8 codes each) make one 16-byte chunk
#pragma unroll
                    for (int i = 0; i < 2; ++i)
                        *reinterpret_cast<uint4*>(bst + chunk_off[2 * q + i]) =
                            make_uint4(operand_word<LV>(w[2 * i], 0), operand_word<LV>(w[2 * i], 1), operand_word<LV>(w[2 * i + 1], 0),
                                       operand_word<LV>(w[2 * i + 1], 1));
                }
            }
        };

        if (total > 0) set_row(l_tile);
#pragma unroll
        for (int d = 0; d < kFusedDepth; ++d)
            if (static_cast<uint32_t>(d) < total) load(ring[d]);
        bool ok = true;
        for (uint32_t base = 0; base < total && ok; base += kFusedDepth) {
#pragma unroll
            for (int d = 0; d < kFusedDepth; ++d) {
                const uint32_t it = base + d;
                if (it < total && ok) {
                    const int s = it % kGemmStages;
                    if (it >= kGemmStages && !mbar_wait(&empty[s], ((it / kGemmStages) - 1) & 1, 24)) {
                        *fail = 1;
                        ok = false;
                    } else {
                        store(ring[d], smem + s * STAGE + A_BYTES);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> tensor core
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&full[s]);
                        if (it + kFusedDepth < total) load(ring[d]);
                    }
                }
            }
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

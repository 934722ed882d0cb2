// Measurement helpers: the two hardware ceilings that the benchmark reports beside the library's own numbers.
//   hbm_read_kernel   a plain streaming read (128-bit loads, nothing written): the read-only HBM ceiling that a
//                     weight-streaming decode kernel can be compared with (a copy moves half of its bytes as writes)
//   mma_i8_issue_kernel  tcgen05.mma kind::i8 on CTA pairs, issued back to back on operands that stay in shared
//                     memory (no loads in the loop): the rate of the tensor pipe itself, at whatever clock the power
//                     limit allows -- the ceiling of a prefill GEMM that could hide all of its data movement
// Neither is part of the quantized layer.
#pragma once

#include "common.cuh"
#include "prefill.cuh"
#include "prefill_2cta.cuh"

namespace qift {

__global__ void __launch_bounds__(256)
hbm_read_kernel(const uint4* __restrict__ src, size_t n16, unsigned int* __restrict__ sink) {
    uint4 acc = make_uint4(0, 0, 0, 0);
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n16; i += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w)
                         : "l"(src + i + j * stride));
#pragma unroll
        for (int j = 0; j < 4; ++j) acc.x ^= v[j].x, acc.y ^= v[j].y, acc.z ^= v[j].z, acc.w ^= v[j].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldg(src + i);
        acc.x ^= v.x, acc.y ^= v.y, acc.z ^= v.z, acc.w ^= v.w;
    }
    const unsigned int r = acc.x ^ acc.y ^ acc.z ^ acc.w;
    if (r == 0x9e3779b9u && sink) atomicAdd(sink, 1u);  // keeps the loads alive; practically never true
}

constexpr int kCalibThreads = 128;
constexpr size_t kCalibSmem = 1024 + 2 * 16384 + 64;

// One CTA pair per two SMs; the leader issues `kblocks` x 4 MMAs (256 tokens x 256 channels x 32 bytes of K each)
// on one resident stage (this CTA's 128 x 128-byte activation rows and 128 x 128-byte weight rows, filled with a
// pseudo-random pattern so that the datapath toggles as it would on real operands).
__global__ void __launch_bounds__(kCalibThreads, 1)
mma_i8_issue_kernel(int kblocks, uint64_t limit_ns) {
    constexpr uint32_t A_BYTES = 16384, TMEM_COLS = 256;
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(256 >> 3) << 17) |
                               (static_cast<uint32_t>(256 >> 4) << 24);
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* done = reinterpret_cast<uint64_t*>(smem + 2 * A_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool leader = cluster_ctarank() == 0;

    uint32_t h = 0x9e3779b9u * (blockIdx.x * kCalibThreads + threadIdx.x + 1);
    for (int i = threadIdx.x; i < 2 * static_cast<int>(A_BYTES) / 4; i += kCalibThreads) {
        h = h * 1664525u + 1013904223u;
        reinterpret_cast<uint32_t*>(smem)[i] = (h >> 8) & 0x07070707u;  // small values: the accumulators cannot overflow
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x == 0) {
        mbar_init(done, 1);
        mbar_fence_init();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (warp == 1 && lane == 0 && leader) {
        const uint32_t a_addr = smem_u32(smem);
        const uint64_t adesc = make_kmajor_sw128_desc(a_addr), bdesc = make_kmajor_sw128_desc(a_addr + A_BYTES);
        for (int kb = 0; kb < kblocks; ++kb) {
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) tc_mma_i8_pair(tmem_base, adesc + 2 * k4, bdesc + 2 * k4, IDESC, (kb | k4) != 0);
        }
        tc_commit_pair(done);  // arrives in both CTAs once every MMA above has completed
    }
    if (threadIdx.x == 0) mbar_wait(done, 0, 0x7d, limit_ns);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace qift

// C-ABI entry points of the qift library: argument checks on the host, then kernel launches on the
// caller's stream.  Single translation unit; the kernels live in the headers included below.
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "calib.cuh"
#include "common.cuh"
#include "decode.cuh"
#include "decode_tc.cuh"
#include "diag.cuh"
#include "grouped.cuh"
#include "kv4.cuh"
#include "pack.cuh"
#include "prefill.cuh"
#include "prefill_2cta.cuh"
#include "prefill_fused.cuh"
#include "prefill_fused_pair.cuh"
#include "quant_rows.cuh"
#include "rotate_quant.cuh"

namespace qift {
namespace {

// Prefill routes by token count (measured on a LLaMA-3.1-8B layer): up to 128 rows one CTA per tile
// expanding the codes in the kernel; up to 512 rows CTA pairs expanding in the kernel (one expansion
// per 256-token tile); beyond that, expanding once into an int8 scratch and re-reading it wins.
// Grouped decode: from this many token rows on the row-split kernel (128-row items) is the faster one.  Measured
// on 16 LLaMA-2-7B layers, row-split flat in M against K-split at 1 / 2 / 4 rows: MNZ 140 us against 125 / 152 /
// 168 us; INT4 232 against 236 / 239 / 258; PoT 191 against 218 / 215 / 217.
inline int wide_min_m(int lv) { return (lv == QIFT_LEVELS_POT || lv == QIFT_LEVELS_INT3) ? 1 : 2; }
constexpr int kFusedMaxM = 128;
constexpr int kFusedPairMaxM = 512;
// Several products of one activation (qift_forward_multi / qift_linear_multi): from this many token rows on the
// decode-to-int8 CTA-pair GEMM with its segments and decode-ahead warps beats the per-output fused routes (a
// LLaMA-3.1-8B layer at 256 / 512 rows: measured in the benchmark's mid_m block).
constexpr int kMultiPairMinM = 129;
inline int auto_prefill_route(int M) {
    return (M <= kFusedMaxM) ? QIFT_ROUTE_PREFILL : (M <= kFusedPairMaxM) ? QIFT_ROUTE_PREFILL_FUSED_PAIR : QIFT_ROUTE_PREFILL_PAIR;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }
inline bool valid_levels(int lv) { return lv >= QIFT_LEVELS_MNZ && lv <= QIFT_LEVELS_INT3; }
// K a whole number of packed words (three-bit codes: of high words, 32 codes each)
inline bool whole_words(int K, int lv) { return K % (lv == QIFT_LEVELS_INT3 ? 32 : codes_per_word(lv)) == 0; }

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the
// stream drains; every kernel here executes griddepcontrol.wait before touching caller memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Opt a kernel in to more than 48 KiB of dynamic shared memory; remembered per kernel so that the
// steady state (and any stream capture after a warm-up call) makes no attribute call.
// The same for a kernel that runs as clusters of two CTAs along x.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), unsigned cluster_x, dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                               Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_pairs(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    return launch_pdl_cluster(kernel, 2u, grid, block, smem, st, std::forward<Args>(args)...);
}

// Host-side caches are keyed by the current device and guarded by one mutex: the shared-memory opt-in
// is an attribute of a kernel in ONE context, and grids are sized for the device that runs them.
constexpr int kMaxDevices = 64;
inline std::mutex& cache_mutex() {
    static std::mutex m;
    return m;
}
inline int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
    return dev;
}

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes) {
    if (bytes <= 32 * 1024) return cudaSuccess;  // static shared memory counts against the 48 KiB default too
    struct Entry {
        const void* fn;
        int dev;
        size_t bytes;
    };
    constexpr int kEntries = 256;
    static Entry table[kEntries];
    static int used = 0;
    const void* key = reinterpret_cast<const void*>(kernel);
    const int dev = current_device();
    std::lock_guard<std::mutex> lock(cache_mutex());
    Entry* slot = nullptr;
    for (int i = 0; i < used; ++i)
        if (table[i].fn == key && table[i].dev == dev) slot = &table[i];
    if (slot && bytes <= slot->bytes) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    if (e != cudaSuccess) return e;
    if (!slot && used < kEntries) slot = &table[used++], slot->fn = key, slot->dev = dev;
    if (slot) slot->bytes = bytes;
    return e;
}

inline int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return QIFT_OK;
    std::fprintf(stderr, "qift: CUDA error: %s\n", cudaGetErrorString(e));
    return QIFT_ERR_CUDA;
}

float inv_sqrt_block(int B) { return static_cast<float>(1.0 / std::sqrt(static_cast<double>(B))); }

int check_rotation_shape(int K, int had_block, bool allow_none) {
    if (K <= 0 || K % 16 != 0 || K > kMaxRowK) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (had_block == 0) return allow_none ? QIFT_OK : QIFT_ERR_UNSUPPORTED_SHAPE;
    if (had_block == K && K % 28 == 0 && is_pow2(K / 28) && K / 28 >= 16) return QIFT_OK;  // H_28 (x) H_{K/28}
    if (had_block < 2 || !is_pow2(had_block) || K % had_block != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;
    return QIFT_OK;
}

int sm_count();

// ------------------------------------------------------------------------------ quantizer, rows in registers
template <bool BF16, bool UPPER, int MID, int R2>
int launch_quantize_rows_as(const void* X, int M, int K, int s0, float clip, float inv_sqrt_b, int8_t* q_a, float* s_a,
                            cudaStream_t st) {
    auto kernel = quantize_rows_kernel<BF16, UPPER, MID, R2>;
    const int threads = ((K / 32) + 31) & ~31;
    const size_t smem = R2 > 0 ? padded_row_bytes(K) : 0;
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    // persistent CTAs: as many as fit the SMs (64 registers per thread, the row in shared memory), rows dealt round-robin
    int per_sm = 2048 / threads;
    if (per_sm > 65536 / (64 * threads)) per_sm = 65536 / (64 * threads);
    if (per_sm > static_cast<int>((220 * 1024) / (smem + 1024))) per_sm = static_cast<int>((220 * 1024) / (smem + 1024));
    if (per_sm < 1) per_sm = 1;
    if (per_sm > 16) per_sm = 16;
    int grid = per_sm * sm_count();
    if (grid > M) grid = M;
    return cuda_status(launch_pdl(kernel, dim3(grid), dim3(threads), smem, st, X, M, K, s0, clip,
                                  inv_sqrt_b, q_a, s_a));
}
template <bool BF16, bool UPPER>
int launch_quantize_rows_bu(const void* X, int M, int K, int had_block, float clip, float inv_sqrt_b, int8_t* q_a, float* s_a,
                            cudaStream_t st) {
    int log_b = 0;
    while ((2 << log_b) <= had_block) ++log_b;      // log2 of the block (0 without rotation)
    const int s0 = log_b < 5 ? log_b : 5, r = log_b - s0;
#define QIFT_ROWS(MID, R2) return launch_quantize_rows_as<BF16, UPPER, MID, R2>(X, M, K, s0, clip, inv_sqrt_b, q_a, s_a, st)
    switch (r) {
        case 0: QIFT_ROWS(0, 0);
        case 1: QIFT_ROWS(0, 1);
        case 2: QIFT_ROWS(0, 2);
        case 3: QIFT_ROWS(0, 3);
        case 4: QIFT_ROWS(0, 4);
        case 5: QIFT_ROWS(1, 1);
        case 6: QIFT_ROWS(1, 2);
        case 7: QIFT_ROWS(1, 3);
        default: QIFT_ROWS(1, 4);
    }
#undef QIFT_ROWS
}
int launch_quantize_rows(const void* X, bool bf16, int M, int K, int had_block, float clip, float inv_sqrt_b, int8_t* q_a, float* s_a,
                         cudaStream_t st) {
    const bool upper_only = clip >= 0.825f;  // |u| / s_u < 8.5: the clamp at -8 cannot act
    if (bf16)
        return upper_only ? launch_quantize_rows_bu<true, true>(X, M, K, had_block, clip, inv_sqrt_b, q_a, s_a, st)
                          : launch_quantize_rows_bu<true, false>(X, M, K, had_block, clip, inv_sqrt_b, q_a, s_a, st);
    return upper_only ? launch_quantize_rows_bu<false, true>(X, M, K, had_block, clip, inv_sqrt_b, q_a, s_a, st)
                      : launch_quantize_rows_bu<false, false>(X, M, K, had_block, clip, inv_sqrt_b, q_a, s_a, st);
}

// ---------------------------------------------------------------------------------------- decode
template <int LV, int NT, int RT>
int launch_decode(const DecodeParams& p, cudaStream_t st) {
    const int words = p.K / codes_per_word(LV);
    const int nchunks = (words + kChunkWords - 1) / kChunkWords;
    const size_t stage = decode_stage_bytes(LV, RT, p.M);
    int stages = static_cast<int>((80 * 1024) / stage);
    if (stages < 2) stages = 2;
    if (stages > nchunks) stages = nchunks;
    DecodeParams q = p;
    q.stages = stages;
    const size_t smem = decode_smem_bytes(LV, RT, NT, p.M, stages);
    auto kernel = linear_decode_kernel<LV, NT, RT>;
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int grid = (p.N + 16 * RT - 1) / (16 * RT);
    return cuda_status(launch_pdl(kernel, dim3(grid), dim3(kDecThreads), smem, st, q));
}

template <int LV>
int dispatch_decode(const DecodeParams& p, cudaStream_t st) {
    if (p.M > 8) return launch_decode<LV, 2, 1>(p, st);
    const int tiles = (p.N + 15) / 16;
    if (tiles >= 4 * 148) return launch_decode<LV, 1, 2>(p, st);
    return launch_decode<LV, 1, 1>(p, st);
}

bool decode_supports(int lv, int M, int N, int K) {
    const int per = codes_per_word(lv);
    return lv != QIFT_LEVELS_INT3 && M >= 1 && M <= 16 && K % (16 * per) == 0;  // whole 16-word warp slices
}

template <int LV>
int launch_generic(const uint32_t* packed, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N, int K,
                   void* Y, int y_bf16, int32_t* acc_debug, cudaStream_t st) {
    const int grid = (N + kGenericWarps - 1) / kGenericWarps;
    return cuda_status(launch_pdl(linear_generic_kernel<LV>, dim3(grid), dim3(kGenericWarps * 32), 0, st, packed, s_n, q_a,
                                  s_a, M, N, K, Y, y_bf16, acc_debug));
}

// --------------------------------------------------------------------------------------- prefill
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// int8 [rows, K] row-major; box = 128 bytes of K x box_rows rows, 128-byte swizzle, zero fill.
bool make_i8_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kGemmBK), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int count[kMaxDevices] = {};
    const int dev = current_device();
    std::lock_guard<std::mutex> lock(cache_mutex());
    if (!count[dev]) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        count[dev] = n > 0 ? n : 148;
    }
    return count[dev];
}

template <int BN>
int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const GemmParams& gp, cudaStream_t st) {
    auto kernel = gemm_i8_tcgen05_kernel<BN>;
    const size_t smem = gemm_smem_bytes<BN>();
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int tiles = ((gp.M + kGemmBM - 1) / kGemmBM) * ((gp.N + BN - 1) / BN);
    const int grid = tiles < sm_count() ? tiles : sm_count();
    return cuda_status(launch_pdl(kernel, dim3(grid), dim3(kGemmThreads), smem, st, ma, mb, gp));
}

template <int LV>
int launch_expand(const uint32_t* packed, int N, int K, int8_t* out, cudaStream_t st) {
    const int row_blocks = (N + kExpandRows - 1) / kExpandRows;
    const int blocks = row_blocks < 148 * 16 ? row_blocks : 148 * 16;   // blocks of rows are dealt to the CTAs
    const int words = K / codes_per_word(LV);
    const int threads = words >= 256 ? 256 : ((words + 31) / 32) * 32;   // short rows: no idle warps
    return cuda_status(launch_pdl(expand_levels_kernel<LV>, dim3(static_cast<unsigned>(blocks)), dim3(threads), 0, st, packed, N,
                                  words, out));
}

// Tile width of the CTA-pair kernels: the one whose rounds over the SM pairs cost least.  Measured at
// M = 2048, K = 4096 a round of 128 / 224 / 256-wide tiles takes 10.3 / 13.0 / 13.5 us (the activation
// tile is re-read from L2 for every channel tile, so narrow tiles are not proportionally cheaper):
// cost ~ width + 284.  14336 channels then run 7 full rounds of 224-wide tiles instead of the
// 6.05 -> 7 rounds of 256-wide ones; 1024 channels one round of 128-wide tiles.
int pair_tile_width(int M, const int* N, int count) {
    const int widths[3] = {256, 224, 128};
    const int pair_count = sm_count() / 2, m_pairs = (M + 2 * kGemmBM - 1) / (2 * kGemmBM);
    int bn = 256;
    long best = -1;
    for (int w : widths) {
        long tiles = 0;
        for (int i = 0; i < count; ++i) tiles += static_cast<long>(m_pairs) * ((N[i] + w - 1) / w);
        const long cost = ((tiles + pair_count - 1) / pair_count) * (w + 284);
        if (best < 0 || cost < best) best = cost, bn = w;
    }
    return bn;
}
inline int pair_tile_width(int M, int N) { return pair_tile_width(M, &N, 1); }

// Host description of one launch of the CTA-pair GEMM: up to kPairMaxSegments products that share the
// activations, and up to kPairMaxSegments side jobs (codes of a later product decoded meanwhile).
struct PairCall {
    const int8_t* q_a;
    const float* s_a;
    int M, K, y_bf16;
    int nseg;
    struct {
        const int8_t* wexp;  // int8 [N, K]
        const float* s_n;
        void* Y;
        int32_t* acc_debug;
        int N;
    } seg[kPairMaxSegments];
    int njobs;
    struct {
        const uint32_t* packed;
        int8_t* out;
        int N, K, levels;
    } job[kPairMaxJobs];
    uint64_t wait_limit_ns;
    int starve;
};

template <int BN>
int launch_gemm_pairs(const PairParams& pp, int tiles, cudaStream_t st) {
    auto kernel = gemm_i8_pair_kernel<BN>;
    const size_t smem = pair_smem_bytes<BN>();
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    int pairs = sm_count() / 2;
    if (pairs > tiles && pp.units == 0) pairs = tiles;  // with side jobs every SM takes its share of them
    return cuda_status(launch_pdl_pairs(kernel, dim3(2 * pairs), dim3(kPairThreads), smem, st, pp));
}

int run_pair_gemm(const PairCall& c, cudaStream_t st) {
    if (c.nseg < 1 || c.nseg > kPairMaxSegments || c.njobs < 0 || c.njobs > kPairMaxJobs) return QIFT_ERR_INVALID_ARG;
    PairParams pp = {};
    int widths[kPairMaxSegments];
    for (int i = 0; i < c.nseg; ++i) widths[i] = c.seg[i].N;
    const int bn = pair_tile_width(c.M, widths, c.nseg);
    if (!make_i8_map(&pp.map_a, c.q_a, c.M, c.K, kGemmBM)) return QIFT_ERR_CUDA;
    int tiles = 0;
    for (int i = 0; i < c.nseg; ++i) {
        // each CTA of a pair loads its own 128 tokens and half of the tile's channels
        if (!make_i8_map(&pp.map_b[i], c.seg[i].wexp, c.seg[i].N, c.K, bn / 2)) return QIFT_ERR_CUDA;
        pp.seg[i] = PairSegment{c.seg[i].s_n, c.seg[i].Y, c.seg[i].acc_debug, c.seg[i].N, tiles};
        tiles += (c.seg[i].N + bn - 1) / bn;
    }
    pp.s_a = c.s_a, pp.M = c.M, pp.K = c.K, pp.y_bf16 = c.y_bf16, pp.nseg = c.nseg, pp.n_tiles = tiles;
    pp.wait_limit_ns = c.wait_limit_ns, pp.starve = c.starve;
    int units = 0;
    for (int i = 0; i < c.njobs; ++i) {
        const int words = c.job[i].K / codes_per_word(c.job[i].levels);
        pp.job[i] = SideJob{c.job[i].packed, c.job[i].out, c.job[i].N, words, units, c.job[i].levels};
        units += ((c.job[i].N + kSideUnitRows - 1) / kSideUnitRows) * ((words + kSideUnitWords - 1) / kSideUnitWords);
    }
    pp.njobs = c.njobs, pp.units = units;
    const int all_tiles = ((c.M + 2 * kGemmBM - 1) / (2 * kGemmBM)) * tiles;
    switch (bn) {
        case 256: return launch_gemm_pairs<256>(pp, all_tiles, st);
        case 224: return launch_gemm_pairs<224>(pp, all_tiles, st);
        default: return launch_gemm_pairs<128>(pp, all_tiles, st);
    }
}

int run_expand(const uint32_t* packed, int lv, int N, int K, int8_t* wexp, cudaStream_t st) {
    switch (lv) {
        case QIFT_LEVELS_MNZ: return launch_expand<QIFT_LEVELS_MNZ>(packed, N, K, wexp, st);
        case QIFT_LEVELS_POT: return launch_expand<QIFT_LEVELS_POT>(packed, N, K, wexp, st);
        case QIFT_LEVELS_SYM: return launch_expand<QIFT_LEVELS_SYM>(packed, N, K, wexp, st);
        case QIFT_LEVELS_INT3: return launch_expand<QIFT_LEVELS_INT3>(packed, N, K, wexp, st);
        default: return launch_expand<QIFT_LEVELS_INT4>(packed, N, K, wexp, st);
    }
}

int run_i8_gemm(const int8_t* wexp, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N, int K, void* Y,
                int y_bf16, int32_t* acc_debug, cudaStream_t st, bool pairs);

int run_prefill(const uint32_t* packed, const float* s_n, int lv, const int8_t* q_a, const float* s_a, int M, int N, int K,
                void* Y, int y_bf16, int32_t* acc_debug, void* workspace, size_t workspace_bytes, cudaStream_t st,
                bool pairs = false) {
    if (K % 16 != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;  // TMA row pitch must be a multiple of 16 bytes
    const size_t need = (static_cast<size_t>(N) * K + 1023) & ~static_cast<size_t>(1023);
    if (!workspace || workspace_bytes < need) return QIFT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    int8_t* wexp = static_cast<int8_t*>(workspace);
    const int rc = run_expand(packed, lv, N, K, wexp, st);
    if (rc != QIFT_OK) return rc;
    return run_i8_gemm(wexp, s_n, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, st, pairs);
}

int run_i8_gemm(const int8_t* wexp, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N, int K, void* Y,
                int y_bf16, int32_t* acc_debug, cudaStream_t st, bool pairs) {
    const int m_tiles = (M + kGemmBM - 1) / kGemmBM;
    const bool narrow = m_tiles * ((N + 255) / 256) < sm_count();
    if (pairs) {
        PairCall c = {};
        c.q_a = q_a, c.s_a = s_a, c.M = M, c.K = K, c.y_bf16 = y_bf16, c.nseg = 1;
        c.seg[0].wexp = wexp, c.seg[0].s_n = s_n, c.seg[0].Y = Y, c.seg[0].acc_debug = acc_debug, c.seg[0].N = N;
        return run_pair_gemm(c, st);
    }
    CUtensorMap ma, mb;
    GemmParams gp{s_n, s_a, Y, acc_debug, M, N, K, y_bf16};
    if (!make_i8_map(&ma, q_a, M, K, kGemmBM) || !make_i8_map(&mb, wexp, N, K, narrow ? 128 : 256)) return QIFT_ERR_CUDA;
    return narrow ? launch_gemm<128>(ma, mb, gp, st) : launch_gemm<256>(ma, mb, gp, st);
}

template <int LV, int BN>
int launch_fused(const CUtensorMap& ma, const FusedParams& fp, cudaStream_t st) {
    auto kernel = gemm_fused_kernel<LV, BN>;
    const size_t smem = fused_smem_bytes<BN>();
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int tiles = ((fp.M + kGemmBM - 1) / kGemmBM) * ((fp.N + BN - 1) / BN);
    const int grid = tiles < sm_count() ? tiles : sm_count();
    return cuda_status(launch_pdl(kernel, dim3(grid), dim3(kFusedThreads), smem, st, ma, fp));
}

template <int LV>
int dispatch_fused(const CUtensorMap& ma, const FusedParams& fp, cudaStream_t st) {
    const int m_tiles = (fp.M + kGemmBM - 1) / kGemmBM;
    const bool narrow = m_tiles * ((fp.N + 255) / 256) < sm_count();
    return narrow ? launch_fused<LV, 128>(ma, fp, st) : launch_fused<LV, 256>(ma, fp, st);
}

template <int LV, int BN>
int launch_fused_pairs(const CUtensorMap& ma, const FusedParams& fp, cudaStream_t st) {
    auto kernel = gemm_fused_pair_kernel<LV, BN>;
    const size_t smem = fused_pair_smem_bytes<BN>();
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    const int tiles = ((fp.M + 2 * kGemmBM - 1) / (2 * kGemmBM)) * ((fp.N + BN - 1) / BN);
    int pairs = sm_count() / 2;
    if (pairs > tiles) pairs = tiles;
    return cuda_status(launch_pdl_pairs(kernel, dim3(2 * pairs), dim3(kFusedThreads), smem, st, ma, fp));
}

template <int LV>
int dispatch_fused_pairs(const CUtensorMap& ma, const FusedParams& fp, cudaStream_t st) {
    switch (pair_tile_width(fp.M, fp.N)) {
        case 256: return launch_fused_pairs<LV, 256>(ma, fp, st);
        case 224: return launch_fused_pairs<LV, 224>(ma, fp, st);
        default: return launch_fused_pairs<LV, 128>(ma, fp, st);
    }
}

// Prefill route with the expansion fused into the GEMM; workspace = per-token sums of q_a.
int run_prefill_fused(const uint32_t* packed, const float* s_n, int lv, const int8_t* q_a, const float* s_a, int M, int N,
                      int K, void* Y, int y_bf16, int32_t* acc_debug, void* workspace, size_t workspace_bytes, cudaStream_t st,
                      bool pairs = false) {
    if (K % 16 != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;  // TMA row pitch must be a multiple of 16 bytes
    const size_t need = (static_cast<size_t>(M) * 4 + 1023) & ~static_cast<size_t>(1023);
    if (!workspace || workspace_bytes < need) return QIFT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    int* sumq = static_cast<int*>(workspace);
    int rc = cuda_status(launch_pdl(rowsum_q_kernel, dim3((M + 7) / 8), dim3(256), 0, st, q_a, M, K, sumq));
    if (rc != QIFT_OK) return rc;
    CUtensorMap ma;
    if (!make_i8_map(&ma, q_a, M, K, kGemmBM)) return QIFT_ERR_CUDA;
    FusedParams fp{packed, s_n, s_a, sumq, Y, acc_debug, M, N, K, y_bf16};
    if (pairs) {
        switch (lv) {
            case QIFT_LEVELS_MNZ: return dispatch_fused_pairs<QIFT_LEVELS_MNZ>(ma, fp, st);
            case QIFT_LEVELS_POT: return dispatch_fused_pairs<QIFT_LEVELS_POT>(ma, fp, st);
            case QIFT_LEVELS_SYM: return dispatch_fused_pairs<QIFT_LEVELS_SYM>(ma, fp, st);
            default: return dispatch_fused_pairs<QIFT_LEVELS_INT4>(ma, fp, st);
        }
    }
    switch (lv) {
        case QIFT_LEVELS_MNZ: return dispatch_fused<QIFT_LEVELS_MNZ>(ma, fp, st);
        case QIFT_LEVELS_POT: return dispatch_fused<QIFT_LEVELS_POT>(ma, fp, st);
        case QIFT_LEVELS_SYM: return dispatch_fused<QIFT_LEVELS_SYM>(ma, fp, st);
        default: return dispatch_fused<QIFT_LEVELS_INT4>(ma, fp, st);
    }
}

// Scratch of QIFT_ROUTE_DECODE_ROWS: the re-laid-out activations and the token sums.
inline size_t decode_rows_scratch(int M, int K) { return ((static_cast<size_t>(M) * K + 255) & ~static_cast<size_t>(255)) + 512; }
// Grouped plans: the row-split mma.sync kernel up to 32 token rows, the tcgen05 weight-streaming kernel from 33 to 128,
// where it is the faster one (a LLaMA-3.1-8B layer, MNZ: 29.5 against 25 us at 32 rows; config 3 at 64 rows: 2.5 against
// 1.7 TB/s for the standard set, 2.3 against 1.5 for PoT).
inline bool tc_rows_applies(int lv, int M) { return lv != QIFT_LEVELS_INT3 && M > 32 && M <= kGroupMaxM; }
inline int tc_tokens(int M) { return M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128; }   // the tensor-core N of that kernel
inline int tc_rows_per_item(int M, int lv) { return kTcRows * tc_tiles_per_item(tc_tokens(M), codes_per_word(lv)); }
constexpr int kInt3MaxRows = 16;   // three-bit codes on the row-split kernel: six accumulator sets per token tile, two token tiles
inline bool decode_rows_supports(int lv, int M, int N, int K) {
    if (lv == QIFT_LEVELS_INT3) return M >= 1 && M <= kInt3MaxRows && K % 256 == 0;
    return M >= 2 && M <= kWideMaxM && decode_supports(lv, M > 16 ? 16 : M, N, K);
}
int run_decode_rows(const uint32_t* packed, const float* s_n, int lv, const int8_t* q_a, const float* s_a, int M, int N, int K,
                    void* Y, int y_bf16, int32_t* acc_debug, void* workspace, cudaStream_t st);
int run_forward_rows(const void* X, int x_bf16, int M, int K, int had_block, float clip, const uint32_t* packed, const float* s_n,
                     int lv, int N, void* Y, int y_bf16, int8_t* q_scratch, float* s_a, int* sumq, cudaStream_t st);

int linear_impl(const uint32_t* packed, const float* s_n, int lv, const int8_t* q_a, const float* s_a, int M, int N, int K,
                void* Y, int y_dtype, int32_t* acc_debug, void* workspace, size_t workspace_bytes, int route, void* stream) {
    if (!packed || !s_n || !q_a || !s_a || !Y || M <= 0 || N <= 0 || K <= 0 || !valid_levels(lv)) return QIFT_ERR_INVALID_ARG;
    if (y_dtype != QIFT_F32 && y_dtype != QIFT_BF16) return QIFT_ERR_INVALID_ARG;
    if (route < QIFT_ROUTE_AUTO || route > QIFT_ROUTE_DECODE_ROWS) return QIFT_ERR_INVALID_ARG;
    if (!whole_words(K, lv) || K % 4 != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(packed) || !aligned16(s_n) || !aligned16(q_a) || !aligned16(s_a) || !aligned16(Y) ||
        (acc_debug && !aligned16(acc_debug)))
        return QIFT_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int y_bf16 = (y_dtype == QIFT_BF16);
    if (lv == QIFT_LEVELS_INT3) {
        // three-bit codes: the row-split decode kernel (from one token row), the decode-to-int8 GEMMs, the generic kernel
        const bool ws_aligned = workspace && (reinterpret_cast<uintptr_t>(workspace) & 255u) == 0;
        if (route == QIFT_ROUTE_AUTO) {
            if (decode_rows_supports(lv, M, N, K) && ws_aligned && workspace_bytes >= decode_rows_scratch(M, K)) route = QIFT_ROUTE_DECODE_ROWS;
            else if (M > kInt3MaxRows && K % 16 == 0) route = (M <= kFusedPairMaxM) ? QIFT_ROUTE_PREFILL_SCRATCH : QIFT_ROUTE_PREFILL_PAIR;
            else route = QIFT_ROUTE_GENERIC;
        }
        if (route == QIFT_ROUTE_DECODE || route == QIFT_ROUTE_PREFILL || route == QIFT_ROUTE_PREFILL_FUSED_PAIR)
            return QIFT_ERR_UNSUPPORTED_SHAPE;
    }
    if (route == QIFT_ROUTE_AUTO) {
        if (M <= 16) {
            route = decode_supports(lv, M, N, K) ? QIFT_ROUTE_DECODE : QIFT_ROUTE_GENERIC;
            // the row-split kernel when the caller brought its scratch (qift_workspace_bytes asks for it); with at most
            // 8 token rows and a small matrix its second launch costs more than it saves (4096 x 4096 at 4 rows: 5.5
            // against 5.2 us; 14336 x 4096: 6.3 against 9.9 us)
            const bool pays = M > 8 || static_cast<long long>(N) * K >= (1ll << 25);
            if (pays && decode_rows_supports(lv, M, N, K) && workspace && workspace_bytes >= decode_rows_scratch(M, K) &&
                (reinterpret_cast<uintptr_t>(workspace) & 255u) == 0)
                route = QIFT_ROUTE_DECODE_ROWS;
        } else {
            route = (K % 16 != 0) ? QIFT_ROUTE_GENERIC : auto_prefill_route(M);
            // 17..64 token rows: still a row-split kernel when its scratch was passed
            if (decode_rows_supports(lv, M, N, K) && workspace && workspace_bytes >= decode_rows_scratch(M, K) &&
                (reinterpret_cast<uintptr_t>(workspace) & 255u) == 0)
                route = QIFT_ROUTE_DECODE_ROWS;
        }
    }
    if (route == QIFT_ROUTE_DECODE_ROWS) {
        if (!decode_rows_supports(lv, M, N, K)) return QIFT_ERR_UNSUPPORTED_SHAPE;
        if (!workspace || workspace_bytes < decode_rows_scratch(M, K)) return QIFT_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(workspace) & 255u) return QIFT_ERR_ALIGNMENT;
        return run_decode_rows(packed, s_n, lv, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, workspace, st);
    }
    if (route == QIFT_ROUTE_DECODE) {
        if (!decode_supports(lv, M, N, K)) return QIFT_ERR_UNSUPPORTED_SHAPE;
        DecodeParams p{packed, s_n, q_a, s_a, Y, acc_debug, M, N, K, y_bf16, 0};
        switch (lv) {
            case QIFT_LEVELS_MNZ: return dispatch_decode<QIFT_LEVELS_MNZ>(p, st);
            case QIFT_LEVELS_POT: return dispatch_decode<QIFT_LEVELS_POT>(p, st);
            case QIFT_LEVELS_SYM: return dispatch_decode<QIFT_LEVELS_SYM>(p, st);
            default: return dispatch_decode<QIFT_LEVELS_INT4>(p, st);
        }
    }
    if (route == QIFT_ROUTE_PREFILL || route == QIFT_ROUTE_PREFILL_FUSED_PAIR)
        return run_prefill_fused(packed, s_n, lv, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, workspace, workspace_bytes, st,
                                 route == QIFT_ROUTE_PREFILL_FUSED_PAIR);
    if (route == QIFT_ROUTE_PREFILL_SCRATCH || route == QIFT_ROUTE_PREFILL_PAIR)
        return run_prefill(packed, s_n, lv, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, workspace, workspace_bytes, st,
                           route == QIFT_ROUTE_PREFILL_PAIR);
    switch (lv) {
        case QIFT_LEVELS_MNZ: return launch_generic<QIFT_LEVELS_MNZ>(packed, s_n, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, st);
        case QIFT_LEVELS_POT: return launch_generic<QIFT_LEVELS_POT>(packed, s_n, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, st);
        case QIFT_LEVELS_SYM: return launch_generic<QIFT_LEVELS_SYM>(packed, s_n, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, st);
        case QIFT_LEVELS_INT3: return launch_generic<QIFT_LEVELS_INT3>(packed, s_n, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, st);
        default: return launch_generic<QIFT_LEVELS_INT4>(packed, s_n, q_a, s_a, M, N, K, Y, y_bf16, acc_debug, st);
    }
}

}  // namespace
}  // namespace qift

using namespace qift;

extern "C" {

const char* qift_status_string(int status) {
    switch (status) {
        case QIFT_OK: return "ok";
        case QIFT_ERR_INVALID_ARG: return "invalid argument";
        case QIFT_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case QIFT_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case QIFT_ERR_WORKSPACE: return "workspace missing or too small";
        case QIFT_ERR_CUDA: return "CUDA error";
        case QIFT_ERR_TIMEOUT: return "device-side wait timed out";
        case QIFT_ERR_TOO_LARGE: return "N*K exceeds the built-in static scratch";
        default: return "unknown status";
    }
}

size_t qift_packed_bytes(int N, int K, int levels) {
    if (N <= 0 || K <= 0 || !valid_levels(levels) || !whole_words(K, levels)) return 0;
    return static_cast<size_t>(round_up16(N)) * packed_pitch(K, levels) * (tile_word_bytes(levels) / 16);
}

size_t qift_workspace_bytes_route(int M, int N, int K, int levels, int route) {
    if (M <= 0 || N <= 0 || K <= 0 || !valid_levels(levels)) return 0;
    size_t b = 0;
    if (levels == QIFT_LEVELS_INT3 && route == QIFT_ROUTE_AUTO)
        route = decode_rows_supports(levels, M, N, K) ? QIFT_ROUTE_DECODE_ROWS : (M <= kInt3MaxRows) ? QIFT_ROUTE_GENERIC : QIFT_ROUTE_PREFILL_PAIR;
    if (route == QIFT_ROUTE_AUTO) {
        route = (M <= 16) ? QIFT_ROUTE_DECODE : auto_prefill_route(M);
        if (decode_rows_supports(levels, M, N, K)) b = decode_rows_scratch(M, K);  // enough for the fallback route as well
    }
    if (route == QIFT_ROUTE_DECODE_ROWS) b = decode_rows_scratch(M, K);
    if ((route == QIFT_ROUTE_PREFILL || route == QIFT_ROUTE_PREFILL_FUSED_PAIR) && b < static_cast<size_t>(M) * 4) b = static_cast<size_t>(M) * 4;
    if (route == QIFT_ROUTE_PREFILL_SCRATCH || route == QIFT_ROUTE_PREFILL_PAIR) b = static_cast<size_t>(N) * K;
    return (b + 1023) & ~static_cast<size_t>(1023);
}

size_t qift_workspace_bytes(int M, int N, int K, int levels) {
    return qift_workspace_bytes_route(M, N, K, levels, QIFT_ROUTE_AUTO);
}

int qift_pack_weights(const float* W, int N, int K, int levels, int scale_mode, float* s_n, uint32_t* packed, void* stream) {
    if (!W || !s_n || !packed || N <= 0 || K <= 0 || !valid_levels(levels)) return QIFT_ERR_INVALID_ARG;
    if (scale_mode < QIFT_SCALE_GIVEN || scale_mode > QIFT_SCALE_MSE) return QIFT_ERR_INVALID_ARG;
    if (K % 16 != 0 || !whole_words(K, levels) || K > kMaxRowK) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(W) || !aligned16(s_n) || !aligned16(packed)) return QIFT_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = static_cast<size_t>(K) * 5;  // the fp32 row and one code byte per weight
#define QIFT_PACK_CASE(LV)                                                                                   \
    case LV: {                                                                                               \
        cudaError_t e = allow_smem(pack_weights_kernel<LV>, smem);                                           \
        if (e != cudaSuccess) return cuda_status(e);                                                         \
        return cuda_status(launch_pdl(pack_weights_kernel<LV>, dim3(round_up16(N)), dim3(kPackThreads), smem, st, W, \
                                      N, K, scale_mode, s_n, packed));                                       \
    }
    switch (levels) {
        QIFT_PACK_CASE(QIFT_LEVELS_MNZ)
        QIFT_PACK_CASE(QIFT_LEVELS_POT)
        QIFT_PACK_CASE(QIFT_LEVELS_SYM)
        QIFT_PACK_CASE(QIFT_LEVELS_INT4)
        QIFT_PACK_CASE(QIFT_LEVELS_INT3)
    }
#undef QIFT_PACK_CASE
    return QIFT_ERR_INVALID_ARG;
}

int qift_unpack_codes(const uint32_t* packed, int N, int K, int levels, uint8_t* codes, void* stream) {
    if (!packed || !codes || N <= 0 || K <= 0 || !valid_levels(levels)) return QIFT_ERR_INVALID_ARG;
    if (!whole_words(K, levels)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(packed) || !aligned16(codes)) return QIFT_ERR_ALIGNMENT;
    const long long total = static_cast<long long>(N) * K;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    return cuda_status(launch_pdl(unpack_codes_kernel, dim3(static_cast<unsigned>(blocks)), dim3(256), 0,
                                  static_cast<cudaStream_t>(stream), packed, total, K, codes_per_word(levels),
                                  levels == QIFT_LEVELS_INT3 ? 1 : 0, codes));
}

int qift_rotate(const float* X, int M, int K, int had_block, float* Y, void* stream) {
    if (!X || !Y || M <= 0 || K <= 0) return QIFT_ERR_INVALID_ARG;
    const int rc = check_rotation_shape(K, had_block, false);
    if (rc != QIFT_OK) return rc;
    if (!aligned16(X) || !aligned16(Y)) return QIFT_ERR_ALIGNMENT;
    const size_t smem = padded_row_bytes(K);
    auto kernel = is_pow2(had_block) ? rotate_rows_kernel<false> : rotate_rows_kernel<true>;
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    return cuda_status(launch_pdl(kernel, dim3(M), dim3(row_threads(K)), smem, static_cast<cudaStream_t>(stream), X, K, had_block,
                                  inv_sqrt_block(had_block), Y));
}

int qift_quantize_act(const void* X, int x_dtype, int M, int K, int had_block, float clip_ratio, int8_t* q_a, float* s_a,
                      void* stream) {
    if (!X || !q_a || !s_a || M <= 0 || K <= 0) return QIFT_ERR_INVALID_ARG;
    if (x_dtype != QIFT_F32 && x_dtype != QIFT_BF16) return QIFT_ERR_INVALID_ARG;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return QIFT_ERR_INVALID_ARG;
    const int rc = check_rotation_shape(K, had_block, true);
    if (rc != QIFT_OK) return rc;
    if (!aligned16(X) || !aligned16(q_a) || !aligned16(s_a)) return QIFT_ERR_ALIGNMENT;
    const float r = had_block > 1 ? inv_sqrt_block(had_block) : 1.0f;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = padded_row_bytes(K);
    if (quantize_rows_supports(K, had_block))  // every element in one thread's registers between passes
        return launch_quantize_rows(X, x_dtype == QIFT_BF16, M, K, had_block, clip_ratio, r, q_a, s_a, st);
    const bool kron = had_block > 1 && !is_pow2(had_block);
    auto kernel = (x_dtype == QIFT_BF16) ? (kron ? quantize_act_kernel<true, true> : quantize_act_kernel<true, false>)
                                         : (kron ? quantize_act_kernel<false, true> : quantize_act_kernel<false, false>);
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    return cuda_status(launch_pdl(kernel, dim3(M), dim3(row_threads(K)), smem, st, X, K, had_block, clip_ratio, r, q_a, s_a));
}

int qift_w2a4_linear(const uint32_t* packed, const float* s_n, int levels, const int8_t* q_a, const float* s_a, int M, int N,
                     int K, void* Y, int y_dtype, int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream) {
    if (levels != QIFT_LEVELS_MNZ && levels != QIFT_LEVELS_POT && levels != QIFT_LEVELS_SYM) return QIFT_ERR_INVALID_ARG;
    return linear_impl(packed, s_n, levels, q_a, s_a, M, N, K, Y, y_dtype, acc_debug, workspace, workspace_bytes,
                       QIFT_ROUTE_AUTO, stream);
}

int qift_w4a4_linear(const uint32_t* packed, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N, int K,
                     void* Y, int y_dtype, int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream) {
    return linear_impl(packed, s_n, QIFT_LEVELS_INT4, q_a, s_a, M, N, K, Y, y_dtype, acc_debug, workspace, workspace_bytes,
                       QIFT_ROUTE_AUTO, stream);
}

int qift_w3a4_linear(const uint32_t* packed, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N, int K,
                     void* Y, int y_dtype, int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream) {
    return linear_impl(packed, s_n, QIFT_LEVELS_INT3, q_a, s_a, M, N, K, Y, y_dtype, acc_debug, workspace, workspace_bytes,
                       QIFT_ROUTE_AUTO, stream);
}

int qift_linear_route(const uint32_t* packed, const float* s_n, int levels, const int8_t* q_a, const float* s_a, int M, int N,
                      int K, void* Y, int y_dtype, int32_t* acc_debug, void* workspace, size_t workspace_bytes, int route,
                      void* stream) {
    return linear_impl(packed, s_n, levels, q_a, s_a, M, N, K, Y, y_dtype, acc_debug, workspace, workspace_bytes, route, stream);
}

namespace {
struct ForwardLayout {
    size_t x_off, q_off, sa_off, y_off, ws_off, total;
};
inline size_t up1k(size_t v) { return (v + 1023) & ~static_cast<size_t>(1023); }
ForwardLayout forward_layout(int M, int N, int K, int levels, int x_dtype, int y_dtype) {
    ForwardLayout L;
    size_t o = 0;
    L.x_off = o, o += up1k(static_cast<size_t>(M) * K * (x_dtype == QIFT_BF16 ? 2 : 4));
    L.q_off = o, o += up1k(static_cast<size_t>(M) * K);
    L.sa_off = o, o += up1k(static_cast<size_t>(M) * 4);
    L.y_off = o, o += up1k(static_cast<size_t>(M) * N * (y_dtype == QIFT_BF16 ? 2 : 4));
    L.ws_off = o, o += qift_workspace_bytes(M, N, K, levels);
    L.total = o;
    return L;
}
}  // namespace

size_t qift_forward_scratch_bytes(int M, int N, int K, int levels, int x_dtype, int y_dtype) {
    if (M <= 0 || N <= 0 || K <= 0 || !valid_levels(levels)) return 0;
    return forward_layout(M, N, K, levels, x_dtype, y_dtype).total;
}

static int forward_impl(const void* X, bool host, int x_dtype, int M, int K, int had_block, float clip_ratio,
                        const uint32_t* packed, const float* s_n, int levels, int N, void* Y, int y_dtype, void* scratch,
                        size_t scratch_bytes, void* stream) {
    if (!X || !Y || !packed || !s_n || M <= 0 || N <= 0 || K <= 0 || !valid_levels(levels)) return QIFT_ERR_INVALID_ARG;
    if ((x_dtype != QIFT_F32 && x_dtype != QIFT_BF16) || (y_dtype != QIFT_F32 && y_dtype != QIFT_BF16))
        return QIFT_ERR_INVALID_ARG;
    if (!whole_words(K, levels)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    const int rs = check_rotation_shape(K, had_block, true);
    if (rs != QIFT_OK) return rs;
    const ForwardLayout L = forward_layout(M, N, K, levels, x_dtype, y_dtype);
    if (!scratch || scratch_bytes < L.total) return QIFT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* base = static_cast<unsigned char*>(scratch);
    const void* x_dev = X;
    void* y_dev = Y;
    if (host) {
        x_dev = base + L.x_off;
        y_dev = base + L.y_off;
        cudaError_t e = cudaMemcpyAsync(base + L.x_off, X, static_cast<size_t>(M) * K * (x_dtype == QIFT_BF16 ? 2 : 4),
                                        cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    int8_t* q_a = reinterpret_cast<int8_t*>(base + L.q_off);
    float* s_a = reinterpret_cast<float*>(base + L.sa_off);
    int rc;
    if (decode_rows_supports(levels, M, N, K) && L.total - L.ws_off >= 512) {
        // 2..64 token rows: the grouped path's quantizer writes the row-split kernel's activation layout directly
        rc = run_forward_rows(x_dev, x_dtype == QIFT_BF16, M, K, had_block, clip_ratio, packed, s_n, levels, N, y_dev,
                              y_dtype == QIFT_BF16, q_a, s_a, reinterpret_cast<int*>(base + L.ws_off), st);
    } else {
        rc = qift_quantize_act(x_dev, x_dtype, M, K, had_block, clip_ratio, q_a, s_a, stream);
        if (rc != QIFT_OK) return rc;
        rc = linear_impl(packed, s_n, levels, q_a, s_a, M, N, K, y_dev, y_dtype, nullptr, base + L.ws_off, L.total - L.ws_off,
                         QIFT_ROUTE_AUTO, stream);
    }
    if (rc != QIFT_OK) return rc;
    if (host) {
        cudaError_t e = cudaMemcpyAsync(Y, y_dev, static_cast<size_t>(M) * N * (y_dtype == QIFT_BF16 ? 2 : 4),
                                        cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return cuda_status(e);
    }
    return QIFT_OK;
}

int qift_forward(const void* X, int x_dtype, int M, int K, int had_block, float clip_ratio, const uint32_t* packed,
                 const float* s_n, int levels, int N, void* Y, int y_dtype, void* scratch, size_t scratch_bytes, void* stream) {
    if (X && !aligned16(X)) return QIFT_ERR_ALIGNMENT;
    if (Y && !aligned16(Y)) return QIFT_ERR_ALIGNMENT;
    return forward_impl(X, false, x_dtype, M, K, had_block, clip_ratio, packed, s_n, levels, N, Y, y_dtype, scratch,
                        scratch_bytes, stream);
}

int qift_forward_host(const void* X_host, int x_dtype, int M, int K, int had_block, float clip_ratio, const uint32_t* packed,
                      const float* s_n, int levels, int N, void* Y_host, int y_dtype, void* scratch, size_t scratch_bytes,
                      void* stream) {
    return forward_impl(X_host, true, x_dtype, M, K, had_block, clip_ratio, packed, s_n, levels, N, Y_host, y_dtype, scratch,
                        scratch_bytes, stream);
}

// ------------------------------------------------------------------------- several products of one activation
namespace {
struct MultiLayout {
    size_t q_off, sa_off, ws_off, total;
};
bool multi_outputs_ok(const qift_linear_output* o, int count, bool need_all) {
    if (!o || count < 1 || count > kPairMaxSegments) return false;
    for (int i = 0; i < count; ++i) {
        if (!o[i].packed || o[i].N <= 0) return false;
        if (need_all && (!o[i].s_n || !o[i].Y)) return false;
    }
    return true;
}
MultiLayout multi_layout(int M, int K, int levels, const qift_linear_output* o, int count) {
    MultiLayout L;
    size_t off = 0;
    L.q_off = off, off += up1k(static_cast<size_t>(M) * K);
    L.sa_off = off, off += up1k(static_cast<size_t>(M) * 4);
    size_t ws = 0;
    if (M < kMultiPairMinM)  // the routes below the pair GEMM bring their own (small) workspace needs
        for (int i = 0; i < count; ++i) {
            const size_t w = qift_workspace_bytes(M, o[i].N, K, levels);
            if (w > ws) ws = w;
        }
    L.ws_off = off, off += ws;
    L.total = off;
    return L;
}
inline size_t levels_offset(int K, const qift_linear_output* o, int i) {  // of output i inside a levels buffer
    size_t off = 0;
    for (int j = 0; j < i; ++j) off += up1k(static_cast<size_t>(o[j].N) * K);
    return off;
}
}  // namespace

size_t qift_levels_bytes(int K, const qift_linear_output* outputs, int count) {
    if (K <= 0 || !multi_outputs_ok(outputs, count, false)) return 0;
    return levels_offset(K, outputs, count);
}

size_t qift_forward_multi_scratch_bytes(int M, int K, int levels, const qift_linear_output* outputs, int count) {
    if (M <= 0 || K <= 0 || !valid_levels(levels) || !multi_outputs_ok(outputs, count, false)) return 0;
    return multi_layout(M, K, levels, outputs, count).total;
}

static int check_outputs_and_ahead(int M, int K, int levels, const qift_linear_output* outputs, int count, int y_dtype,
                                   const qift_decode_ahead* ahead) {
    if (M <= 0 || K <= 0 || !valid_levels(levels) || !multi_outputs_ok(outputs, count, true)) return QIFT_ERR_INVALID_ARG;
    if (y_dtype != QIFT_F32 && y_dtype != QIFT_BF16) return QIFT_ERR_INVALID_ARG;
    if (!whole_words(K, levels)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    for (int i = 0; i < count; ++i)
        if (!aligned16(outputs[i].packed) || !aligned16(outputs[i].s_n) || !aligned16(outputs[i].Y) ||
            (outputs[i].acc_debug && !aligned16(outputs[i].acc_debug)))
            return QIFT_ERR_ALIGNMENT;
    int ahead_outputs = 0;
    for (const qift_decode_ahead* a = ahead; a; a = a->next) {
        if (!multi_outputs_ok(a->outputs, a->count, false) || a->K <= 0 || !valid_levels(a->levels) || !a->levels_buf)
            return QIFT_ERR_INVALID_ARG;
        if ((ahead_outputs += a->count) > kPairMaxJobs) return QIFT_ERR_INVALID_ARG;
        if (a->K % 16 != 0 || !whole_words(a->K, a->levels)) return QIFT_ERR_UNSUPPORTED_SHAPE;
        if (a->levels_bytes < qift_levels_bytes(a->K, a->outputs, a->count)) return QIFT_ERR_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(a->levels_buf) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
        for (int i = 0; i < a->count; ++i)
            if (!aligned16(a->outputs[i].packed)) return QIFT_ERR_ALIGNMENT;
    }
    return QIFT_OK;
}

// S4 + S5 for every output on one quantized activation; arguments checked by the callers.
static int linear_multi_impl(const int8_t* q_a, const float* s_a, int M, int K, int levels, const qift_linear_output* outputs, int count,
                             int y_dtype, void* workspace, size_t workspace_bytes, void* levels_buf, size_t levels_bytes,
                             int levels_ready, const qift_decode_ahead* ahead, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool pair_route = M >= kMultiPairMinM && K % 16 == 0;
    int rc;
    if (!pair_route) {
        for (int i = 0; i < count; ++i) {
            rc = linear_impl(outputs[i].packed, outputs[i].s_n, levels, q_a, s_a, M, outputs[i].N, K, outputs[i].Y, y_dtype,
                             outputs[i].acc_debug, workspace, workspace_bytes, QIFT_ROUTE_AUTO, stream);
            if (rc != QIFT_OK) return rc;
        }
        for (const qift_decode_ahead* a = ahead; a; a = a->next)
            for (int i = 0; i < a->count; ++i) {
                int8_t* out = static_cast<int8_t*>(a->levels_buf) + levels_offset(a->K, a->outputs, i);
                rc = run_expand(a->outputs[i].packed, a->levels, a->outputs[i].N, a->K, out, st);
                if (rc != QIFT_OK) return rc;
            }
        return QIFT_OK;
    }
    if (!levels_buf || levels_bytes < qift_levels_bytes(K, outputs, count)) return QIFT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(levels_buf) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    PairCall c = {};
    c.q_a = q_a, c.s_a = s_a, c.M = M, c.K = K, c.y_bf16 = (y_dtype == QIFT_BF16), c.nseg = count;
    for (int i = 0; i < count; ++i) {
        int8_t* wexp = static_cast<int8_t*>(levels_buf) + levels_offset(K, outputs, i);
        if (!levels_ready) {
            rc = run_expand(outputs[i].packed, levels, outputs[i].N, K, wexp, st);
            if (rc != QIFT_OK) return rc;
        }
        c.seg[i].wexp = wexp, c.seg[i].s_n = outputs[i].s_n, c.seg[i].Y = outputs[i].Y, c.seg[i].acc_debug = outputs[i].acc_debug;
        c.seg[i].N = outputs[i].N;
    }
    // the side warps decode one-plane layouts; three-bit codes are decoded by separate launches after the GEMM
    for (const qift_decode_ahead* a = ahead; a; a = a->next) {
        if (a->levels == QIFT_LEVELS_INT3) continue;
        for (int i = 0; i < a->count; ++i) {
            auto& j = c.job[c.njobs++];
            j.packed = a->outputs[i].packed, j.N = a->outputs[i].N, j.K = a->K, j.levels = a->levels;
            j.out = static_cast<int8_t*>(a->levels_buf) + levels_offset(a->K, a->outputs, i);
        }
    }
    rc = run_pair_gemm(c, st);
    if (rc != QIFT_OK) return rc;
    for (const qift_decode_ahead* a = ahead; a; a = a->next) {
        if (a->levels != QIFT_LEVELS_INT3) continue;
        for (int i = 0; i < a->count; ++i) {
            int8_t* out = static_cast<int8_t*>(a->levels_buf) + levels_offset(a->K, a->outputs, i);
            rc = run_expand(a->outputs[i].packed, a->levels, a->outputs[i].N, a->K, out, st);
            if (rc != QIFT_OK) return rc;
        }
    }
    return QIFT_OK;
}

size_t qift_linear_multi_workspace_bytes(int M, int K, int levels, const qift_linear_output* outputs, int count) {
    if (M <= 0 || K <= 0 || !valid_levels(levels) || !multi_outputs_ok(outputs, count, false)) return 0;
    const MultiLayout L = multi_layout(M, K, levels, outputs, count);
    return L.total - L.ws_off;
}

int qift_linear_multi(const int8_t* q_a, const float* s_a, int M, int K, int levels, const qift_linear_output* outputs, int count,
                      int y_dtype, void* workspace, size_t workspace_bytes, void* levels_buf, size_t levels_bytes, int levels_ready,
                      const qift_decode_ahead* ahead, void* stream) {
    if (!q_a || !s_a) return QIFT_ERR_INVALID_ARG;
    const int rc = check_outputs_and_ahead(M, K, levels, outputs, count, y_dtype, ahead);
    if (rc != QIFT_OK) return rc;
    if (!aligned16(q_a) || !aligned16(s_a)) return QIFT_ERR_ALIGNMENT;
    if (workspace_bytes < qift_linear_multi_workspace_bytes(M, K, levels, outputs, count) || (workspace_bytes && !workspace))
        return QIFT_ERR_WORKSPACE;
    if (workspace && (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    return linear_multi_impl(q_a, s_a, M, K, levels, outputs, count, y_dtype, workspace, workspace_bytes, levels_buf, levels_bytes,
                             levels_ready, ahead, stream);
}

int qift_forward_multi(const void* X, int x_dtype, int M, int K, int had_block, float clip_ratio, int levels,
                       const qift_linear_output* outputs, int count, int y_dtype, void* scratch, size_t scratch_bytes,
                       void* levels_buf, size_t levels_bytes, int levels_ready, const qift_decode_ahead* ahead, void* stream) {
    if (!X || (x_dtype != QIFT_F32 && x_dtype != QIFT_BF16)) return QIFT_ERR_INVALID_ARG;
    int rc = check_outputs_and_ahead(M, K, levels, outputs, count, y_dtype, ahead);
    if (rc != QIFT_OK) return rc;
    if (!aligned16(X)) return QIFT_ERR_ALIGNMENT;
    const MultiLayout L = multi_layout(M, K, levels, outputs, count);
    if (!scratch || scratch_bytes < L.total) return QIFT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    if (M >= kMultiPairMinM && K % 16 == 0) {  // found before anything is launched
        if (!levels_buf || levels_bytes < qift_levels_bytes(K, outputs, count)) return QIFT_ERR_WORKSPACE;
        if ((reinterpret_cast<uintptr_t>(levels_buf) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    }
    unsigned char* base = static_cast<unsigned char*>(scratch);
    int8_t* q_a = reinterpret_cast<int8_t*>(base + L.q_off);
    float* s_a = reinterpret_cast<float*>(base + L.sa_off);
    rc = qift_quantize_act(X, x_dtype, M, K, had_block, clip_ratio, q_a, s_a, stream);
    if (rc != QIFT_OK) return rc;
    return linear_multi_impl(q_a, s_a, M, K, levels, outputs, count, y_dtype, base + L.ws_off, L.total - L.ws_off, levels_buf,
                             levels_bytes, levels_ready, ahead, stream);
}

// ------------------------------------------------------------------------------------------- grouped
// Plan layout: header, problem records, token sums [count][kGroupMaxM], then (128-byte aligned) one tensor map per
// problem over its q_a, which the tcgen05 kernel's activation loads use.
static size_t plan_maps_offset(int count) {
    const size_t o = sizeof(GroupHeader) + static_cast<size_t>(count) * (sizeof(GroupProblemDev) + kGroupMaxM * sizeof(int));
    return (o + 127) & ~static_cast<size_t>(127);
}
size_t qift_group_plan_bytes(int count) {
    if (count <= 0) return 0;
    return plan_maps_offset(count) + static_cast<size_t>(count) * sizeof(CUtensorMap);
}

int qift_group_plan(const qift_group_problem* problems, int count, int M, int levels, int x_dtype, int y_dtype, float clip_ratio,
                    void* plan_host, void* plan_dev, size_t plan_bytes, void* stream) {
    if (!problems || !plan_host || !plan_dev || count <= 0 || M <= 0 || !valid_levels(levels)) return QIFT_ERR_INVALID_ARG;
    if ((x_dtype != QIFT_F32 && x_dtype != QIFT_BF16) || (y_dtype != QIFT_F32 && y_dtype != QIFT_BF16))
        return QIFT_ERR_INVALID_ARG;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return QIFT_ERR_INVALID_ARG;
    if (M > kGroupMaxM || (levels == QIFT_LEVELS_INT3 && M > kInt3MaxRows)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (M > kWideMaxM && !tc_rows_applies(levels, M)) return QIFT_ERR_UNSUPPORTED_SHAPE;   // 65 .. 128 rows: the tcgen05 kernel only
    if (plan_bytes < qift_group_plan_bytes(count)) return QIFT_ERR_WORKSPACE;
    if (!aligned16(plan_dev) || !aligned16(plan_host)) return QIFT_ERR_ALIGNMENT;
    if (tc_rows_applies(levels, M) && (reinterpret_cast<uintptr_t>(plan_dev) & 127u) != 0) return QIFT_ERR_ALIGNMENT;  // tensor maps
    // Rows per work item, which also selects the kernel (dispatch_grouped): 64 / 32 for the K-split kernel, 128 for the
    // row-split kernel, 256 (two row tiles per warp, with two token tiles) when that still leaves two items per SM.
    int rows_per_item = (M >= wide_min_m(levels)) ? kWideRows : 64;  // below wide_min_m there is only M = 1
    const bool use_tc = tc_rows_applies(levels, M);                  // 33 .. 64 rows (not PoT): the tcgen05 kernel, 256-row items
    if (use_tc) rows_per_item = tc_rows_per_item(M, levels);
    // (INT4 only: PoT measured slower with two tiles per warp, and the two-bit sets are faster as two CTAs per SM of 128-row
    // items -- config 3 at 16 rows: 4.27 against 4.07 TB/s)
    if (!use_tc && rows_per_item == kWideRows && M > 8 && M <= 16 && levels == QIFT_LEVELS_INT4) {
        long long items256 = 0;
        for (int i = 0; i < count; ++i) items256 += (problems[i].N + 2 * kWideRows - 1) / (2 * kWideRows);
        if (items256 >= 2ll * sm_count()) rows_per_item = 2 * kWideRows;
    }
    GroupHeader* h = static_cast<GroupHeader*>(plan_host);
    GroupProblemDev* d = reinterpret_cast<GroupProblemDev*>(h + 1);
    int items = 0, max_k = 0, any_kron = 0;
    for (int i = 0; i < count; ++i) {
        const qift_group_problem& q = problems[i];
        if (!q.X || !q.packed || !q.s_n || !q.q_a || !q.s_a || !q.Y || q.N <= 0 || q.K <= 0) return QIFT_ERR_INVALID_ARG;
        if (levels == QIFT_LEVELS_INT3 ? !decode_rows_supports(levels, M, q.N, q.K) : !decode_supports(levels, M > 16 ? 16 : M, q.N, q.K))
            return QIFT_ERR_UNSUPPORTED_SHAPE;
        const int rs = check_rotation_shape(q.K, q.had_block, true);
        if (rs != QIFT_OK) return rs;
        if (!aligned16(q.X) || !aligned16(q.packed) || !aligned16(q.s_n) || !aligned16(q.q_a) || !aligned16(q.s_a) ||
            !aligned16(q.Y) || (q.acc_debug && !aligned16(q.acc_debug)))
            return QIFT_ERR_ALIGNMENT;
        GroupProblemDev& o = d[i];
        o.X = q.X, o.packed = q.packed, o.s_n = q.s_n, o.q_a = q.q_a, o.s_a = q.s_a, o.Y = q.Y, o.acc_debug = q.acc_debug;
        o.N = q.N, o.K = q.K, o.had_block = q.had_block;
        o.item_begin = items;
        o.inv_sqrt_b = q.had_block > 1 ? inv_sqrt_block(q.had_block) : 1.0f;
        o.quant_src = i;
        for (int j = 0; j < i; ++j)
            if (d[j].X == q.X && d[j].q_a == q.q_a && d[j].s_a == q.s_a && d[j].K == q.K && d[j].had_block == q.had_block) {
                o.quant_src = d[j].quant_src;
                break;
            }
        for (int j = 0; j < 4; ++j) o.pad[j] = 0;
        items += (q.N + rows_per_item - 1) / rows_per_item;
        if (q.K > max_k) max_k = q.K;
        if (q.had_block > 1 && !is_pow2(q.had_block)) any_kron = 1;
    }
    *h = GroupHeader{};
    h->magic = kGroupMagic, h->count = count, h->M = M, h->levels = levels, h->y_bf16 = (y_dtype == QIFT_BF16);
    h->x_bf16 = (x_dtype == QIFT_BF16), h->clip = clip_ratio, h->total_items = items, h->rows_per_item = rows_per_item;
    h->max_k = max_k;
    h->any_kron = any_kron;
    // the row-split kernel stages one K-chunk of all tokens per copy: its q_a is chunk-major (ChunkMajorDst)
    h->q_pot_lut = (rows_per_item >= kWideRows && levels == QIFT_LEVELS_POT && M > 8) ? 1 : 0;  // the kernel's POT_LUT (both kernels from 9 rows)
    h->q_chunk_bytes = (rows_per_item >= kWideRows) ? wide_chunk_words(rows_per_item / 16, wide_token_tiles(M), levels) * codes_per_word(levels) : 0;
    h->reserved[0] = use_tc ? 1 : 0;
    if (use_tc) h->q_chunk_bytes = 0;  // that kernel reads q_a row-major (prescaled even planes, as the K-split kernel does)
    cudaError_t ce = cudaMemcpyAsync(plan_dev, plan_host, sizeof(GroupHeader) + static_cast<size_t>(count) * sizeof(GroupProblemDev),
                                     cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess || !use_tc) return cuda_status(ce);
    // the tcgen05 kernel stages a k-block of all token rows with one tensor copy: q_a [M, K] int8, box = 128 bytes of K x its
    // token count (rows beyond M read as zero), 128-byte swizzle -- the layout its B descriptor expects
    CUtensorMap* maps = reinterpret_cast<CUtensorMap*>(static_cast<unsigned char*>(plan_host) + plan_maps_offset(count));
    for (int i = 0; i < count; ++i)
        if (!make_i8_map(&maps[i], d[i].q_a, M, d[i].K, tc_tokens(M))) return QIFT_ERR_CUDA;
    return cuda_status(cudaMemcpyAsync(static_cast<unsigned char*>(plan_dev) + plan_maps_offset(count), maps,
                                       static_cast<size_t>(count) * sizeof(CUtensorMap), cudaMemcpyHostToDevice,
                                       static_cast<cudaStream_t>(stream)));
}

}  // extern "C"

namespace {
const GroupHeader* plan_header(const void* plan_host, const void* plan_dev) {
    if (!plan_host || !plan_dev) return nullptr;
    const GroupHeader* h = static_cast<const GroupHeader*>(plan_host);
    return h->magic == kGroupMagic ? h : nullptr;
}

inline const int* plan_sumq(const void* plan_dev, int count) {
    return reinterpret_cast<const int*>(reinterpret_cast<const GroupProblemDev*>(static_cast<const GroupHeader*>(plan_dev) + 1) +
                                        count);
}

template <int LV, int NT, int RT, bool M1>
int launch_grouped(const GroupHeader* h, const GroupProblemDev* host, const GroupProblemDev* dev, const int* sumq,
                   cudaStream_t st) {
    auto kernel = linear_grouped_kernel<LV, NT, RT, M1>;
    const size_t stage = decode_stage_bytes(LV, RT, h->M) + 16;
    for (int first = 0; first < h->count; first += kGroupSlice) {  // the problem table of a launch lives in shared memory
        const int count = (h->count - first < kGroupSlice) ? h->count - first : kGroupSlice;
        const int item_first = host[first].item_begin;
        const int item_end = (first + count < h->count) ? host[first + count].item_begin : h->total_items;
        const size_t fixed = grouped_fixed_smem(LV, RT, h->M, count);
        constexpr int cps = grouped_ctas_per_sm<LV>();  // each CTA gets its share of the SM's shared memory
        int stages = static_cast<int>(((cps == 2 ? 113 : 226) * 1024 - fixed) / stage);
        if (stages < 2) stages = 2;
        if (stages > 12) stages = 12;
        const size_t smem = grouped_smem_bytes(LV, RT, h->M, stages, count);
        cudaError_t e = allow_smem(kernel, smem);
        if (e != cudaSuccess) return cuda_status(e);
        int grid = cps * sm_count();
        if (grid > item_end - item_first) grid = item_end - item_first;
        GroupParams gp{dev + first, sumq, first, count, item_first, item_end, h->M, h->y_bf16, stages};
        const int rc = cuda_status(launch_pdl(kernel, dim3(grid), dim3(kDecThreads), smem, st, gp));
        if (rc != QIFT_OK) return rc;
    }
    return QIFT_OK;
}

// From this many token rows on: 128- or 256-row items split by rows over the warps, one CTA per SM.
template <int LV, int NT, int RT, int CWARPS>
int launch_grouped_wide(const GroupHeader* h, const GroupProblemDev* host, const GroupProblemDev* dev, const int* sumq,
                        cudaStream_t st, bool single = false) {
    auto kernel = linear_grouped_wide_kernel<LV, NT, RT, CWARPS>;
    const size_t stage = wide_stage_bytes(LV, h->M, RT * CWARPS) + 16;
    for (int first = 0; first < h->count; first += kGroupSlice) {
        const int count = (h->count - first < kGroupSlice) ? h->count - first : kGroupSlice;
        const int item_first = host[first].item_begin;
        const int item_end = (first + count < h->count) ? host[first + count].item_begin : h->total_items;
        constexpr int cps = wide_ctas_per_sm(LV, NT, RT * CWARPS);   // each CTA gets its share of the SM's shared memory
        int stages = static_cast<int>(((cps == 2 ? 112 : 226) * 1024 - static_cast<size_t>(count) * sizeof(SmemProblem) - 64) / stage);
        if (stages < 2) stages = 2;
        if (stages > 8) stages = 8;
        const size_t smem = wide_smem_bytes(LV, h->M, RT * CWARPS, stages, count);
        cudaError_t e = allow_smem(kernel, smem);
        if (e != cudaSuccess) return cuda_status(e);
        int grid = cps * sm_count();
        if (grid > item_end - item_first) grid = item_end - item_first;
        GroupParams gp{dev + first, sumq, first, count, item_first, item_end, h->M, h->y_bf16, stages, 0, {}};
        if (single) gp.use_single = 1, gp.single = host[0];
        const int rc = cuda_status(launch_pdl(kernel, dim3(grid), dim3((CWARPS + 1) * 32), smem, st, gp));
        if (rc != QIFT_OK) return rc;
    }
    return QIFT_OK;
}

// The tcgen05 weight-streaming kernel: 128-channel items, one persistent CTA per SM.  At least 132 KiB of shared memory is
// requested whatever the stage sizes, so that two of these CTAs can never share an SM: each allocates all of tensor memory.
template <int LV, int NTOK>
int launch_tc(const GroupHeader* h, const GroupProblemDev* host, const GroupProblemDev* dev, const int* sumq, cudaStream_t st,
              bool single = false) {
    {
        constexpr int R = tc_tiles_per_item(NTOK, codes_per_word(LV));
        auto kernel = linear_tc_kernel<LV, NTOK, R>;
        for (int first = 0; first < h->count; first += kGroupSlice) {
            const int count = (h->count - first < kGroupSlice) ? h->count - first : kGroupSlice;
            const int item_first = host[first].item_begin;
            const int item_end = (first + count < h->count) ? host[first + count].item_begin : h->total_items;
            size_t smem = tc_smem_bytes(NTOK, count);
            if (smem < 132 * 1024) smem = 132 * 1024;
            cudaError_t e = allow_smem(kernel, smem);
            if (e != cudaSuccess) return cuda_status(e);
            int grid = sm_count();
            if (grid > item_end - item_first) grid = item_end - item_first;
            GroupParams gp{dev + first, sumq, first, count, item_first, item_end, h->M, h->y_bf16, 0, 0, {}};
            if (single) return QIFT_ERR_INVALID_ARG;   // the kernel needs the plan's tensor maps
            // dev points just behind the header of the device plan: the maps follow the token sums
            const unsigned char* plan_dev = reinterpret_cast<const unsigned char*>(dev) - sizeof(GroupHeader);
            gp.maps = reinterpret_cast<const CUtensorMap*>(plan_dev + plan_maps_offset(h->count)) + first;
            const int rc = cuda_status(launch_pdl(kernel, dim3(grid), dim3(kTcThreads), smem, st, gp));
            if (rc != QIFT_OK) return rc;
        }
        return QIFT_OK;
    }
}
template <int LV>
int dispatch_tc(const GroupHeader* h, const GroupProblemDev* host, const GroupProblemDev* dev, const int* sumq, cudaStream_t st,
                bool single = false) {
    switch (tc_tokens(h->M)) {
        case 16: return launch_tc<LV, 16>(h, host, dev, sumq, st, single);
        case 32: return launch_tc<LV, 32>(h, host, dev, sumq, st, single);
        case 64: return launch_tc<LV, 64>(h, host, dev, sumq, st, single);
        default: return launch_tc<LV, 128>(h, host, dev, sumq, st, single);
    }
}

template <int LV>
int dispatch_grouped(const GroupHeader* h, const GroupProblemDev* host, const GroupProblemDev* dev, const int* sumq,
                     cudaStream_t st) {
    if constexpr (LV == QIFT_LEVELS_INT3) {   // three-bit codes: the row-split kernel with one or two token tiles
        if (h->rows_per_item != kWideRows || h->M > kInt3MaxRows) return QIFT_ERR_INVALID_ARG;
        return h->M > 8 ? launch_grouped_wide<LV, 2, 1, 8>(h, host, dev, sumq, st) : launch_grouped_wide<LV, 1, 1, 8>(h, host, dev, sumq, st);
    } else {
    if (h->reserved[0]) return dispatch_tc<LV>(h, host, dev, sumq, st);   // the plan chose the tcgen05 kernel (33 .. 64 rows)
    // (256-row items as sixteen consumer warps were measured slower and are not dispatched.)
    if (h->rows_per_item == 2 * kWideRows) return launch_grouped_wide<LV, 2, 2, 8>(h, host, dev, sumq, st);
    if (h->rows_per_item == kWideRows && h->M > 32) return launch_grouped_wide<LV, 8, 1, 8>(h, host, dev, sumq, st);
    if (h->rows_per_item == kWideRows && h->M > 16) return launch_grouped_wide<LV, 4, 1, 8>(h, host, dev, sumq, st);
    if (h->rows_per_item == kWideRows)
        return h->M > 8 ? launch_grouped_wide<LV, 2, 1, 8>(h, host, dev, sumq, st) : launch_grouped_wide<LV, 1, 1, 8>(h, host, dev, sumq, st);
    if (h->M == 1) return launch_grouped<LV, 1, 4, true>(h, host, dev, sumq, st);
    return QIFT_ERR_INVALID_ARG;  // no plan has other row counts per item
    }
}
}  // namespace

namespace qift {
namespace {
int run_decode_rows(const uint32_t* packed, const float* s_n, int lv, const int8_t* q_a, const float* s_a, int M, int N, int K,
                    void* Y, int y_bf16, int32_t* acc_debug, void* workspace, cudaStream_t st) {
    int8_t* q_out = static_cast<int8_t*>(workspace);
    int* sumq = reinterpret_cast<int*>(q_out + ((static_cast<size_t>(M) * K + 255) & ~static_cast<size_t>(255)));
    // (The tcgen05 kernel serves grouped plans only: one product has too few 256-channel items to fill the SMs -- a
    // LLaMA-3.1-8B layer of seven calls at 64 rows takes 374 us on it against 190 us on this kernel.)
    GroupHeader h{};
    h.magic = kGroupMagic, h.count = 1, h.M = M, h.levels = lv, h.y_bf16 = y_bf16, h.rows_per_item = kWideRows;
    h.total_items = (N + kWideRows - 1) / kWideRows;
    h.q_pot_lut = (lv == QIFT_LEVELS_POT && M > 8) ? 1 : 0;
    h.q_chunk_bytes = wide_chunk_words(kDecWarps, wide_token_tiles(M), lv) * codes_per_word(lv);
    GroupProblemDev rec{};
    rec.X = nullptr, rec.packed = packed, rec.s_n = s_n, rec.q_a = q_out, rec.s_a = const_cast<float*>(s_a), rec.Y = Y;
    rec.acc_debug = acc_debug, rec.N = N, rec.K = K, rec.had_block = 0, rec.item_begin = 0, rec.inv_sqrt_b = 1.0f, rec.quant_src = 0;
    int rc = cuda_status(launch_pdl(relayout_act_kernel, dim3(M), dim3(128), 0, st, q_a, M, K, lv == QIFT_LEVELS_INT4 ? 1 : 0,
                                    h.q_chunk_bytes, h.q_pot_lut, q_out, sumq));
    if (rc != QIFT_OK) return rc;
    const GroupProblemDev* none = nullptr;
#define QIFT_ROWS_CASE(LV)                                                                                          \
    case LV:                                                                                                        \
        return M > 32 ? launch_grouped_wide<LV, 8, 1, 8>(&h, &rec, none, sumq, st, true)                            \
               : M > 16 ? launch_grouped_wide<LV, 4, 1, 8>(&h, &rec, none, sumq, st, true)                          \
               : M > 8 ? launch_grouped_wide<LV, 2, 1, 8>(&h, &rec, none, sumq, st, true)                           \
                       : launch_grouped_wide<LV, 1, 1, 8>(&h, &rec, none, sumq, st, true);
    switch (lv) {
        QIFT_ROWS_CASE(QIFT_LEVELS_MNZ)
        QIFT_ROWS_CASE(QIFT_LEVELS_POT)
        QIFT_ROWS_CASE(QIFT_LEVELS_SYM)
        case QIFT_LEVELS_INT3:
            return M > 8 ? launch_grouped_wide<QIFT_LEVELS_INT3, 2, 1, 8>(&h, &rec, none, sumq, st, true)
                         : launch_grouped_wide<QIFT_LEVELS_INT3, 1, 1, 8>(&h, &rec, none, sumq, st, true);
        default:
            QIFT_ROWS_CASE(QIFT_LEVELS_INT4)
    }
#undef QIFT_ROWS_CASE
}

int run_forward_rows(const void* X, int x_bf16, int M, int K, int had_block, float clip, const uint32_t* packed, const float* s_n,
                     int lv, int N, void* Y, int y_bf16, int8_t* q_scratch, float* s_a, int* sumq, cudaStream_t st) {
    GroupHeader h{};
    h.magic = kGroupMagic, h.count = 1, h.M = M, h.levels = lv, h.y_bf16 = y_bf16, h.rows_per_item = kWideRows;
    h.total_items = (N + kWideRows - 1) / kWideRows;
    h.q_pot_lut = (lv == QIFT_LEVELS_POT && M > 8) ? 1 : 0;
    h.q_chunk_bytes = wide_chunk_words(kDecWarps, wide_token_tiles(M), lv) * codes_per_word(lv);
    GroupProblemDev rec{};
    rec.X = X, rec.packed = packed, rec.s_n = s_n, rec.q_a = q_scratch, rec.s_a = s_a, rec.Y = Y, rec.acc_debug = nullptr;
    rec.N = N, rec.K = K, rec.had_block = had_block, rec.item_begin = 0, rec.quant_src = 0;
    rec.inv_sqrt_b = had_block > 1 ? inv_sqrt_block(had_block) : 1.0f;
    const bool kron = had_block > 1 && !is_pow2(had_block);
    auto qk = x_bf16 ? (kron ? quantize_act_grouped_kernel<true, true> : quantize_act_grouped_kernel<true, false>)
                     : (kron ? quantize_act_grouped_kernel<false, true> : quantize_act_grouped_kernel<false, false>);
    const size_t smem = padded_row_bytes(K);
    cudaError_t e = allow_smem(qk, smem);
    if (e != cudaSuccess) return cuda_status(e);
    const GroupProblemDev* none = nullptr;
    int rc = cuda_status(launch_pdl(qk, dim3(M), dim3(kRowThreads), smem, st, none, sumq, M, clip, lv == QIFT_LEVELS_INT4 ? 1 : 0,
                                    h.q_chunk_bytes, h.q_pot_lut, 1, rec));
    if (rc != QIFT_OK) return rc;
#define QIFT_ROWS_CASE(LV)                                                                                          \
    case LV:                                                                                                        \
        return M > 32 ? launch_grouped_wide<LV, 8, 1, 8>(&h, &rec, none, sumq, st, true)                            \
               : M > 16 ? launch_grouped_wide<LV, 4, 1, 8>(&h, &rec, none, sumq, st, true)                          \
               : M > 8 ? launch_grouped_wide<LV, 2, 1, 8>(&h, &rec, none, sumq, st, true)                           \
                       : launch_grouped_wide<LV, 1, 1, 8>(&h, &rec, none, sumq, st, true);
    switch (lv) {
        QIFT_ROWS_CASE(QIFT_LEVELS_MNZ)
        QIFT_ROWS_CASE(QIFT_LEVELS_POT)
        QIFT_ROWS_CASE(QIFT_LEVELS_SYM)
        case QIFT_LEVELS_INT3:
            return M > 8 ? launch_grouped_wide<QIFT_LEVELS_INT3, 2, 1, 8>(&h, &rec, none, sumq, st, true)
                         : launch_grouped_wide<QIFT_LEVELS_INT3, 1, 1, 8>(&h, &rec, none, sumq, st, true);
        default:
            QIFT_ROWS_CASE(QIFT_LEVELS_INT4)
    }
#undef QIFT_ROWS_CASE
}
}  // namespace
}  // namespace qift

extern "C" {

int qift_group_quantize_act(const void* plan_host, const void* plan_dev, void* stream) {
    const GroupHeader* h = plan_header(plan_host, plan_dev);
    if (!h) return QIFT_ERR_INVALID_ARG;
    const GroupProblemDev* dev = reinterpret_cast<const GroupProblemDev*>(static_cast<const GroupHeader*>(plan_dev) + 1);
    const size_t smem = padded_row_bytes(h->max_k);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* sumq = const_cast<int*>(plan_sumq(plan_dev, h->count));
    const dim3 grid(static_cast<unsigned>(h->count) * h->M);
    const bool kron = h->any_kron != 0;  // some problem uses the full-dimension rotation: the variant with the 28-point pass
    auto kernel = h->x_bf16 ? (kron ? quantize_act_grouped_kernel<true, true> : quantize_act_grouped_kernel<true, false>)
                            : (kron ? quantize_act_grouped_kernel<false, true> : quantize_act_grouped_kernel<false, false>);
    cudaError_t e = allow_smem(kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    return cuda_status(launch_pdl(kernel, grid, dim3(kRowThreads), smem, st, dev, sumq, h->M, h->clip,
                                  h->levels == QIFT_LEVELS_INT4 ? 1 : 0, h->q_chunk_bytes, h->q_pot_lut, 0, GroupProblemDev{}));
}

int qift_group_linear(const void* plan_host, const void* plan_dev, void* stream) {
    const GroupHeader* h = plan_header(plan_host, plan_dev);
    if (!h) return QIFT_ERR_INVALID_ARG;
    const GroupProblemDev* dev = reinterpret_cast<const GroupProblemDev*>(static_cast<const GroupHeader*>(plan_dev) + 1);
    const GroupProblemDev* host = reinterpret_cast<const GroupProblemDev*>(h + 1);
    const int* sumq = plan_sumq(plan_dev, h->count);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    switch (h->levels) {
        case QIFT_LEVELS_MNZ: return dispatch_grouped<QIFT_LEVELS_MNZ>(h, host, dev, sumq, st);
        case QIFT_LEVELS_POT: return dispatch_grouped<QIFT_LEVELS_POT>(h, host, dev, sumq, st);
        case QIFT_LEVELS_SYM: return dispatch_grouped<QIFT_LEVELS_SYM>(h, host, dev, sumq, st);
        case QIFT_LEVELS_INT3: return dispatch_grouped<QIFT_LEVELS_INT3>(h, host, dev, sumq, st);
        default: return dispatch_grouped<QIFT_LEVELS_INT4>(h, host, dev, sumq, st);
    }
}

int qift_group_forward(const void* plan_host, const void* plan_dev, void* stream) {
    const int rc = qift_group_quantize_act(plan_host, plan_dev, stream);
    if (rc != QIFT_OK) return rc;
    return qift_group_linear(plan_host, plan_dev, stream);
}

int qift_group_forward_host(const void* plan_host, const void* plan_dev, const void* x_host, void* x_dev, size_t x_bytes,
                            const void* y_dev, void* y_host, size_t y_bytes, void* stream) {
    if (!x_host || !x_dev || !y_dev || !y_host || x_bytes == 0 || y_bytes == 0) return QIFT_ERR_INVALID_ARG;
    if (!plan_header(plan_host, plan_dev)) return QIFT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_status(e);
    const int rc = qift_group_forward(plan_host, plan_dev, stream);
    if (rc != QIFT_OK) return rc;
    return cuda_status(cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, st));
}

// ------------------------------------------------------------------------- allocation-free product
}  // extern "C"

namespace {
// Scratch for the decoded int8 levels of qift_w2a4_linear_static.  In host code this name is only a
// handle for the runtime's symbol lookup, never a device address: kernels get the address that
// cudaGetSymbolAddress returns.
constexpr size_t kStaticScratchBytes = size_t(16) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

void* g_static_scratch_addr[qift::kMaxDevices] = {};

// Device address of the array on the current device; looked up once per device (primary context, no
// device reset in between).
cudaError_t static_scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= qift::kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(qift::cache_mutex());
    if (!g_static_scratch_addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_scratch_addr[dev] = ptr;
    }
    *out = g_static_scratch_addr[dev];
    return cudaSuccess;
}
}  // namespace

extern "C" {

size_t qift_static_scratch_bytes(void) { return kStaticScratchBytes; }

int qift_w2a4_linear_static(const uint32_t* packed, const float* s_n, int levels, const int8_t* q_a, const float* s_a, int M,
                            int N, int K, void* Y, int y_dtype, int32_t* acc_debug, void* stream) {
    if (levels != QIFT_LEVELS_MNZ && levels != QIFT_LEVELS_POT && levels != QIFT_LEVELS_SYM) return QIFT_ERR_INVALID_ARG;
    if (!packed || !s_n || !q_a || !s_a || !Y || M <= 0 || N <= 0 || K <= 0) return QIFT_ERR_INVALID_ARG;
    if (y_dtype != QIFT_F32 && y_dtype != QIFT_BF16) return QIFT_ERR_INVALID_ARG;
    if (K % 16 != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(packed) || !aligned16(s_n) || !aligned16(q_a) || !aligned16(s_a) || !aligned16(Y) ||
        (acc_debug && !aligned16(acc_debug)))
        return QIFT_ERR_ALIGNMENT;
    if (static_cast<size_t>(N) * static_cast<size_t>(K) > kStaticScratchBytes) {
        std::fprintf(stderr, "qift_w2a4_linear_static: N*K = %zu bytes of scratch needed, the built-in array holds %zu\n",
                     static_cast<size_t>(N) * static_cast<size_t>(K), kStaticScratchBytes);
        return QIFT_ERR_TOO_LARGE;
    }
    void* scratch = nullptr;
    const cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return cuda_status(e);
    return linear_impl(packed, s_n, levels, q_a, s_a, M, N, K, Y, y_dtype, acc_debug, scratch, kStaticScratchBytes,
                       QIFT_ROUTE_PREFILL_SCRATCH, stream);
}

// --------------------------------------------------------------------------------- diagnostics
namespace {

struct RatioScanLayout {
    int seg, V, scan_blocks, chunks;
    size_t P, keys_a, keys_b, hist, digit_totals, block_s1, block_s2, totals, ratios, partial, bytes;
};

bool ratio_scan_layout(long long n, int R, RatioScanLayout& l) {
    if (n < 1 || n > (1ll << 28) || R < 1 || R > 65535) return false;
    long long seg = (n + 4095) / 4096;
    seg = (seg + 31) / 32 * 32;
    if (seg < 1024) seg = 1024;
    l.seg = static_cast<int>(seg);
    l.V = static_cast<int>((n + seg - 1) / seg);
    l.scan_blocks = static_cast<int>((n + kScanBlock - 1) / kScanBlock);
    l.chunks = static_cast<int>((n + 1 + kEvalBlock - 1) / kEvalBlock);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off += (bytes + 255) / 256 * 256;
        return at;
    };
    l.P = take(sizeof(double) * n);
    l.keys_a = take(sizeof(uint32_t) * n);
    l.keys_b = take(sizeof(uint32_t) * n);
    l.hist = take(sizeof(uint32_t) * 256 * l.V);
    l.digit_totals = take(sizeof(uint32_t) * 256);
    l.block_s1 = take(sizeof(double) * l.scan_blocks);
    l.block_s2 = take(sizeof(double) * l.scan_blocks);
    l.totals = take(sizeof(double) * 2);
    l.ratios = take(sizeof(double) * R);
    l.partial = take(sizeof(ScanBest) * static_cast<size_t>(R) * l.chunks);
    l.bytes = off;
    return true;
}

int stream_blocks(long long items) {
    long long blocks = (items + kDiagThreads - 1) / kDiagThreads;
    const long long cap = static_cast<long long>(sm_count()) * 8;
    return static_cast<int>(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}

}  // namespace

int qift_diag_grid_quantize(const float* W, int N, int K, const float* grid, int scale_mode, float* s_n, uint8_t* codes,
                            void* stream) {
    if (!W || !grid || !s_n || N <= 0 || K <= 0) return QIFT_ERR_INVALID_ARG;
    if (scale_mode != QIFT_SCALE_GIVEN && scale_mode != QIFT_SCALE_ABSMAX && scale_mode != QIFT_SCALE_MSE) return QIFT_ERR_INVALID_ARG;
    if (!(grid[0] < grid[1] && grid[1] < grid[2] && grid[2] < grid[3] && grid[3] > 0.0f)) return QIFT_ERR_INVALID_ARG;
    if (K > 16384) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(W)) return QIFT_ERR_ALIGNMENT;
    Grid4 G;
    for (int i = 0; i < 4; ++i) G.g[i] = grid[i];
    for (int i = 0; i < 3; ++i) G.m[i] = (grid[i] + grid[i + 1]) * 0.5f;
    const size_t smem = sizeof(float) * K;
    cudaError_t e = allow_smem(grid_quantize_kernel, smem);
    if (e != cudaSuccess) return cuda_status(e);
    grid_quantize_kernel<<<N, kDiagThreads, smem, static_cast<cudaStream_t>(stream)>>>(W, K, G, scale_mode, s_n, codes);
    return cuda_status(cudaGetLastError());
}

int qift_diag_bucket_stats(const float* W, const uint8_t* codes, int N, int K, const float* s_n, const float* values, int L,
                           unsigned long long* count, double* sqerr, void* stream) {
    if (!W || !codes || !s_n || !values || !count || !sqerr || N <= 0 || K <= 0) return QIFT_ERR_INVALID_ARG;
    if (L != 4 && L != 16) return QIFT_ERR_INVALID_ARG;
    if (K % 4 != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(W) || (reinterpret_cast<uintptr_t>(codes) & 3u) || (reinterpret_cast<uintptr_t>(count) & 7u) ||
        (reinterpret_cast<uintptr_t>(sqerr) & 7u))
        return QIFT_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(count, 0, sizeof(unsigned long long) * L, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(sqerr, 0, sizeof(double) * L, st);
    if (e != cudaSuccess) return cuda_status(e);
    BucketValues v = {};
    for (int i = 0; i < L; ++i) v.v[i] = values[i];
    const long long total4 = static_cast<long long>(N) * K / 4;
    const int blocks = stream_blocks(total4);
    if (L == 4)
        bucket_stats_kernel<4><<<blocks, kDiagThreads, 0, st>>>(W, codes, total4, K, s_n, v, count, sqerr);
    else
        bucket_stats_kernel<16><<<blocks, kDiagThreads, 0, st>>>(W, codes, total4, K, s_n, v, count, sqerr);
    return cuda_status(cudaGetLastError());
}

size_t qift_diag_ratio_scan_workspace_bytes(long long n, int R) {
    RatioScanLayout l;
    return ratio_scan_layout(n, R, l) ? l.bytes : 0;
}

int qift_diag_ratio_scan(const float* x, long long n, const double* ratios, int R, double* beta, double* nmse, void* workspace,
                         size_t workspace_bytes, void* stream) {
    if (!x || !ratios || !beta || !nmse || n <= 0 || R <= 0) return QIFT_ERR_INVALID_ARG;
    for (int i = 0; i < R && i < 65536; ++i)
        if (!(ratios[i] > 0.0 && ratios[i] <= 1.0)) return QIFT_ERR_INVALID_ARG;
    RatioScanLayout l;
    if (!ratio_scan_layout(n, R, l)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!workspace || workspace_bytes < l.bytes) return QIFT_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return QIFT_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    double* P = reinterpret_cast<double*>(ws + l.P);
    uint32_t* keys_a = reinterpret_cast<uint32_t*>(ws + l.keys_a);
    uint32_t* keys_b = reinterpret_cast<uint32_t*>(ws + l.keys_b);
    uint32_t* hist = reinterpret_cast<uint32_t*>(ws + l.hist);
    uint32_t* digit_totals = reinterpret_cast<uint32_t*>(ws + l.digit_totals);
    double* block_s1 = reinterpret_cast<double*>(ws + l.block_s1);
    double* block_s2 = reinterpret_cast<double*>(ws + l.block_s2);
    double* totals = reinterpret_cast<double*>(ws + l.totals);
    double* d_ratios = reinterpret_cast<double*>(ws + l.ratios);
    ScanBest* partial = reinterpret_cast<ScanBest*>(ws + l.partial);

    cudaError_t e = cudaMemcpyAsync(d_ratios, ratios, sizeof(double) * R, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_status(e);
    abs_keys_kernel<<<stream_blocks(n), kDiagThreads, 0, st>>>(x, n, keys_a);
    const int seg_blocks = (l.V + kDiagWarps - 1) / kDiagWarps;
    uint32_t* in = keys_a;
    uint32_t* out = keys_b;
    for (int shift = 0; shift < 32; shift += 8) {  // four stable passes: the sorted keys end in keys_a
        radix_hist_kernel<<<seg_blocks, kDiagThreads, 0, st>>>(in, n, l.seg, l.V, shift, hist);
        radix_rowscan_kernel<<<256, 1024, 0, st>>>(hist, l.V, digit_totals);
        radix_scatter_kernel<<<seg_blocks, kDiagThreads, 0, st>>>(in, n, l.seg, l.V, shift, hist, digit_totals, out);
        uint32_t* t = in;
        in = out;
        out = t;
    }
    scan_block_sums_kernel<<<l.scan_blocks, kDiagThreads, 0, st>>>(keys_a, n, block_s1, block_s2);
    scan_bases_kernel<<<1, kDiagThreads, 0, st>>>(block_s1, block_s2, l.scan_blocks, totals);
    scan_write_kernel<<<l.scan_blocks, kDiagThreads, 0, st>>>(keys_a, n, block_s1, P);
    ratio_eval_kernel<<<dim3(l.chunks, R), kDiagThreads, 0, st>>>(keys_a, P, n, totals, d_ratios, partial);
    ratio_final_kernel<<<R, kDiagThreads, 0, st>>>(partial, l.chunks, totals, beta, nmse);
    return cuda_status(cudaGetLastError());
}

int qift_device_status(void* stream, uint32_t* detail) {
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_status(e);
    unsigned int word = 0;
    e = cudaMemcpyFromSymbol(&word, g_status_word, sizeof(word));
    if (e != cudaSuccess) return cuda_status(e);
    if (detail) *detail = word;
    if (word == 0) return QIFT_OK;
    const unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_status_word, &zero, sizeof(zero));
    if (e != cudaSuccess) return cuda_status(e);
    return QIFT_ERR_TIMEOUT;
}

}  // extern "C"

namespace qift {
constexpr unsigned int kSiteProbe = 0x7e;
// One thread waits, with the given bound, for a phase of an mbarrier that nobody completes.
__global__ void wait_probe_kernel(uint64_t limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(&bar, 0, kSiteProbe, limit_ns);
}
}  // namespace qift

extern "C" int qift_calib_hbm_read(const void* buf, size_t bytes, unsigned int* sink, void* stream) {
    if (!buf || bytes < 16) return QIFT_ERR_INVALID_ARG;
    if (!aligned16(buf)) return QIFT_ERR_ALIGNMENT;
    hbm_read_kernel<<<sm_count() * 8, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint4*>(buf), bytes / 16, sink);
    return cuda_status(cudaGetLastError());
}

extern "C" int qift_calib_mma_i8(int kblocks, double* ops, void* stream) {
    if (kblocks < 1 || kblocks > (1 << 20)) return QIFT_ERR_INVALID_ARG;  // at ~0.3 us per k-block: a third of a second at most
    cudaError_t e = allow_smem(mma_i8_issue_kernel, kCalibSmem);
    if (e != cudaSuccess) return cuda_status(e);
    const int pairs = sm_count() / 2;
    if (ops) *ops = 2.0 * 256 * 256 * 128 * static_cast<double>(kblocks) * pairs;
    return cuda_status(launch_pdl_pairs(mma_i8_issue_kernel, dim3(2 * pairs), dim3(kCalibThreads), kCalibSmem,
                                        static_cast<cudaStream_t>(stream), kblocks, kWaitLimitNs));
}

extern "C" int qift_selftest_wait_timeout(int which, unsigned int limit_us, void* stream) {
    if ((which != 0 && which != 1) || limit_us == 0 || limit_us > 1000000u) return QIFT_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint64_t limit_ns = static_cast<uint64_t>(limit_us) * 1000ull;
    if (which == 0) {
        wait_probe_kernel<<<1, 32, 0, st>>>(limit_ns);
        return cuda_status(cudaGetLastError());
    }
    // The CTA-pair GEMM on one 256 x 256 x 128 tile whose producers issue no loads: the MMA thread's wait for
    // operands and the epilogue warps' wait for the accumulator run out, every role leaves its loop, both CTAs
    // meet at the closing cluster barrier and tensor memory is freed.  Operands live in the built-in scratch;
    // nothing is read or written (no load is issued and no accumulator ever completes).
    void* scratch = nullptr;
    const cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return cuda_status(e);
    unsigned char* base = static_cast<unsigned char*>(scratch);
    PairCall c = {};
    c.q_a = reinterpret_cast<const int8_t*>(base), c.s_a = reinterpret_cast<const float*>(base + 65536);
    c.M = 256, c.K = 128, c.y_bf16 = 1, c.nseg = 1;
    c.seg[0].wexp = reinterpret_cast<const int8_t*>(base + 32768), c.seg[0].s_n = reinterpret_cast<const float*>(base + 69632);
    c.seg[0].Y = base + 131072, c.seg[0].acc_debug = nullptr, c.seg[0].N = 256;
    c.wait_limit_ns = limit_ns, c.starve = 1;
    return run_pair_gemm(c, st);
}

namespace {
// Token splits of the decode attention: one resident wave of CTAs, whole 64-token rounds of the four
// warps per split.
void kv4_splits(int T, int Hkv, int* splits, int* tokens_per_split) {
    int want = (2 * sm_count()) / Hkv;  // two CTAs fit an SM: one resident wave (measured best of 1..4)
    if (want < 1) want = 1;
    int tps = (T + want - 1) / want;
    const int round = kKvTile * kKvWarps;  // tokens the warps of a CTA take per trip
    tps = ((tps + round - 1) / round) * round;
    *tokens_per_split = tps;
    *splits = (T + tps - 1) / tps;  // <= 2 * SMs / Hkv, far below kKvMaxSplits
}
}  // namespace

extern "C" {

int qift_kv4_quantize(const void* X, int x_dtype, int T, int H, int D, int had_block, float clip_ratio, int t0, int T_cap,
                      int layout, uint8_t* codes, float* scale, float* zero, void* stream) {
    if (!X || !codes || !scale || !zero || T <= 0 || H <= 0 || t0 < 0 || T_cap <= 0) return QIFT_ERR_INVALID_ARG;
    if (static_cast<long long>(t0) + T > T_cap) return QIFT_ERR_INVALID_ARG;
    if (x_dtype != QIFT_F32 && x_dtype != QIFT_BF16) return QIFT_ERR_INVALID_ARG;
    if (layout != QIFT_KV_KEYS && layout != QIFT_KV_VALUES) return QIFT_ERR_INVALID_ARG;
    if (!(clip_ratio > 0.0f && clip_ratio <= 1.0f)) return QIFT_ERR_INVALID_ARG;
    if (D != kKvD || (T_cap & 1)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (had_block < 0 || (had_block > 1 && (!is_pow2(had_block) || had_block > D))) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(X) || !aligned16(codes) || !aligned16(scale) || !aligned16(zero)) return QIFT_ERR_ALIGNMENT;
    const float r = had_block > 1 ? inv_sqrt_block(had_block) : 1.0f;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (layout == QIFT_KV_VALUES) {
        const long long warps = static_cast<long long>(((t0 + T + 1) >> 1) - (t0 >> 1)) * H;
        const dim3 grid(static_cast<unsigned>((warps + 7) / 8));
        if (x_dtype == QIFT_BF16)
            return cuda_status(launch_pdl(kv4_quantize_pairs_kernel<true>, grid, dim3(256), 0, st, X, T, H, had_block, r, clip_ratio,
                                          t0, T_cap, codes, scale, zero));
        return cuda_status(launch_pdl(kv4_quantize_pairs_kernel<false>, grid, dim3(256), 0, st, X, T, H, had_block, r, clip_ratio, t0,
                                      T_cap, codes, scale, zero));
    }
    const long long rows = static_cast<long long>(T) * H;
    const dim3 grid(static_cast<unsigned>((rows + 7) / 8));
    if (x_dtype == QIFT_BF16)
        return cuda_status(launch_pdl(kv4_quantize_kernel<true>, grid, dim3(256), 0, st, X, rows, H, had_block, r, clip_ratio, t0,
                                      T_cap, codes, scale, zero));
    return cuda_status(launch_pdl(kv4_quantize_kernel<false>, grid, dim3(256), 0, st, X, rows, H, had_block, r, clip_ratio, t0,
                                  T_cap, codes, scale, zero));
}

int qift_expand_weights(const uint32_t* packed, int N, int K, int levels, int8_t* levels_out, void* stream) {
    if (!packed || !levels_out || N <= 0 || K <= 0 || !valid_levels(levels)) return QIFT_ERR_INVALID_ARG;
    if (K % 16 != 0 || !whole_words(K, levels)) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(packed) || (reinterpret_cast<uintptr_t>(levels_out) & 255u) != 0) return QIFT_ERR_ALIGNMENT;
    return run_expand(packed, levels, N, K, levels_out, static_cast<cudaStream_t>(stream));
}

int qift_expanded_linear(const int8_t* levels_in, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N, int K,
                         void* Y, int y_dtype, int32_t* acc_debug, void* stream) {
    if (!levels_in || !s_n || !q_a || !s_a || !Y || M <= 0 || N <= 0 || K <= 0) return QIFT_ERR_INVALID_ARG;
    if (y_dtype != QIFT_F32 && y_dtype != QIFT_BF16) return QIFT_ERR_INVALID_ARG;
    if (K % 16 != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if ((reinterpret_cast<uintptr_t>(levels_in) & 255u) != 0 || !aligned16(s_n) || !aligned16(q_a) || !aligned16(s_a) ||
        !aligned16(Y) || (acc_debug && !aligned16(acc_debug)))
        return QIFT_ERR_ALIGNMENT;
    return run_i8_gemm(levels_in, s_n, q_a, s_a, M, N, K, Y, y_dtype == QIFT_BF16, acc_debug, static_cast<cudaStream_t>(stream),
                       true);
}

size_t qift_kv4_attention_workspace_bytes(int T, int Hq, int Hkv) {
    if (T <= 0 || Hq <= 0 || Hkv <= 0) return 0;
    int splits, tps;
    kv4_splits(T, Hkv, &splits, &tps);
    return static_cast<size_t>(Hq) * splits * kKvPartial * sizeof(float);
}

int qift_kv4_attention_decode(const float* q, const uint8_t* k_codes, const float* k_scale, const float* k_zero,
                              const uint8_t* v_codes, const float* v_scale, const float* v_zero, int T, int T_cap, int Hq,
                              int Hkv, int D, float* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!q || !k_codes || !k_scale || !k_zero || !v_codes || !v_scale || !v_zero || !out) return QIFT_ERR_INVALID_ARG;
    if (T <= 0 || T > T_cap || Hq <= 0 || Hkv <= 0) return QIFT_ERR_INVALID_ARG;
    if (D != kKvD || Hq % Hkv != 0) return QIFT_ERR_UNSUPPORTED_SHAPE;
    const int G = Hq / Hkv;
    if (G > 8 || (T_cap & 1) || T_cap > (1 << 24)) return QIFT_ERR_UNSUPPORTED_SHAPE;  // 32-bit byte offsets inside a head
    if (!aligned16(q) || !aligned16(k_codes) || !aligned16(v_codes) || !aligned16(k_scale) || !aligned16(k_zero) ||
        !aligned16(v_scale) || !aligned16(v_zero) || !aligned16(out) || !aligned16(workspace))
        return QIFT_ERR_ALIGNMENT;
    Kv4Params p{};
    kv4_splits(T, Hkv, &p.splits, &p.tokens_per_split);
    if (p.splits > kKvMaxSplits) return QIFT_ERR_UNSUPPORTED_SHAPE;
    if (!workspace || workspace_bytes < static_cast<size_t>(Hq) * p.splits * kKvPartial * sizeof(float)) return QIFT_ERR_WORKSPACE;
    p.q = q, p.k_codes = k_codes, p.k_scale = k_scale, p.k_zero = k_zero, p.v_codes = v_codes, p.v_scale = v_scale;
    p.v_zero = v_zero, p.partial = static_cast<float*>(workspace), p.out = out;
    p.T = T, p.T_cap = T_cap, p.Hq = Hq, p.Hkv = Hkv, p.heads_per_kv = G;
    p.inv_sqrt_d = static_cast<float>(1.0 / std::sqrt(static_cast<double>(D)));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rc = cuda_status(launch_pdl(kv4_attention_partial_kernel, dim3(p.splits, p.Hkv), dim3(32 * kKvWarps), 0, st, p));
    if (rc != QIFT_OK) return rc;
    return cuda_status(launch_pdl(kv4_attention_combine_kernel, dim3(p.Hq), dim3(kKvCombineThreads), 0, st, p));
}

}  // extern "C"

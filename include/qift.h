/*
 * qift.h -- C ABI of the B200 (sm_100a) library for the rotated W2A4 / W4A4 quantized linear layer
 * of "Qift: Shift-Friendly No-Zero W2 Post-Training Quantization for Rotated W2A4/KV4 LLM Inference".
 *
 *     y[m,n] = s_n[n] * ( sum_k level(code[n,k]) * q_a[m,k] ) * s_a[m]
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 *   - every pointer is DEVICE memory owned by the caller; the library allocates nothing; base pointers
 *     must be 16-byte aligned.  State the library keeps per process: the device status word (see
 *     qift_device_status), a per-device table of kernels already opted in to large shared memory, the
 *     per-device SM count, and the per-device address of the built-in scratch of
 *     qift_w2a4_linear_static.  The last three assume the primary context of each device and no
 *     cudaDeviceReset while the library is in use;
 *   - all work is enqueued asynchronously on `stream` (a cudaStream_t passed as void*, NULL = the
 *     legacy default stream); nothing synchronizes;
 *   - matrices are row-major with the last index contiguous: W [N,K], X / q_a [M,K], Y [M,N];
 *   - the return value is a qift_status; argument, shape and alignment errors are found on the host
 *     before anything is launched, so a failing call has touched no buffer;
 *   - kernels are launched with programmatic stream serialization: each waits for its predecessor
 *     in the stream before it reads or writes any caller buffer, so ordinary stream order holds.
 *     One exception: the product kernels start fetching the PACKED WEIGHTS before that wait (this is
 *     what lets consecutive layers overlap).  It is safe whenever the weights were written by
 *     qift_pack_weights, by a copy, or by any kernel that does not itself use programmatic early
 *     launch -- i.e. always, unless a caller's own kernel both writes packed weights and calls
 *     cudaTriggerProgrammaticLaunchCompletion before finishing them.
 */
#ifndef QIFT_H_
#define QIFT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QIFT_OK = 0,
    QIFT_ERR_INVALID_ARG = 1,       /* null pointer, non-positive size, unknown enum value          */
    QIFT_ERR_UNSUPPORTED_SHAPE = 2, /* K not a multiple of the codes per word, had_block invalid... */
    QIFT_ERR_ALIGNMENT = 3,         /* a base pointer is not 16-byte aligned                        */
    QIFT_ERR_WORKSPACE = 4,         /* workspace missing or smaller than qift_workspace_bytes()     */
    QIFT_ERR_CUDA = 5,              /* a CUDA runtime call or a launch failed                       */
    QIFT_ERR_TIMEOUT = 6,           /* a bounded device-side wait expired (see qift_device_status)  */
    QIFT_ERR_TOO_LARGE = 7          /* N*K exceeds the built-in scratch of qift_w2a4_linear_static  */
} qift_status;

/* Reconstruction level sets.  Two-bit codes index the levels in ascending order (code 0 = most
 * negative); the paper leaves the code assignment to the implementation (Sec. 3.3). */
typedef enum {
    QIFT_LEVELS_MNZ = 0,  /* {-3,-1,+1,+3}: half-scale form of {+-0.5,+-1.5}; s_n is s/2 (Sec. 3.3) */
    QIFT_LEVELS_POT = 1,  /* {-4,-1,+1,+4}: power-of-two mirror no-zero set          (Sec. 3.3)     */
    QIFT_LEVELS_SYM = 2,  /* {-2,-1, 0,+1}: standard symmetric integer W2            (Eq. 1, b = 2) */
    QIFT_LEVELS_INT4 = 3, /* -8..7 two's-complement nibble, 8 codes per word         (Eq. 1, b = 4) */
    QIFT_LEVELS_INT3 = 4  /* -4..3 two's-complement three-bit code, stored as a two-bit and a one-bit
                             plane: the W3A4 configuration of Sec. 4.4       (Eq. 1, b = 3) */
} qift_levels;

/* How the per-output-channel scale is chosen (Sec. 3.5; the clipping-ratio sweep of Sec. 4.5.1).
 * GIVEN reads s_n; ABSMAX writes s_n = amax / top_level; MSE sweeps the 80 ratios
 * p = 1.00, 0.99, ..., 0.21, s = (p * amax) / top_level, and keeps the first least-squared-error one.
 * The squared errors are fp64 sums whose order of addition is the kernel's: two candidates whose
 * errors agree to 1e-12 relative count as tied, and either may win (a CPU check must allow that and
 * then compare the codes given the returned scale, which are exact).
 * top_level is 3 (MNZ), 4 (POT), 1 (SYM), 7 (INT4), 3 (INT3).  An all-zero row gets s_n = 1. */
typedef enum { QIFT_SCALE_GIVEN = 0, QIFT_SCALE_ABSMAX = 1, QIFT_SCALE_MSE = 2 } qift_scale_mode;

typedef enum { QIFT_F32 = 0, QIFT_BF16 = 1 } qift_dtype;

/* Kernel route of qift_linear_route(): AUTO picks by M. */
typedef enum {
    QIFT_ROUTE_AUTO = 0,
    QIFT_ROUTE_GENERIC = 1,  /* one warp per output channel, dp4a; any M, any K                     */
    QIFT_ROUTE_DECODE = 2,   /* bulk-copy staged, in-register decode, mma.sync; M <= 16             */
    QIFT_ROUTE_PREFILL = 3,  /* tcgen05 kind::i8 GEMM, codes expanded in the kernel; scratch 4*M    */
    QIFT_ROUTE_PREFILL_SCRATCH = 4, /* codes expanded to an int8 [N,K] scratch first, then a TMA-fed
                                      tcgen05 GEMM, one CTA per tile; scratch N*K bytes            */
    QIFT_ROUTE_PREFILL_PAIR = 5,   /* the same with CTA pairs (tcgen05 cta_group::2, 256-token tiles);
                                      scratch N*K bytes                                            */
    QIFT_ROUTE_PREFILL_FUSED_PAIR = 6, /* CTA pairs with the codes expanded in the kernel (each CTA
                                      expands half of the tile's channels); scratch 4*M            */
    QIFT_ROUTE_DECODE_ROWS = 7 /* 2 <= M <= 64: the activations re-laid out into the scratch, then the
                                  row-split kernel of the grouped path (128-row items, no reduction);
                                  scratch M*K + 512 bytes                                         */
} qift_route;

const char* qift_status_string(int status);

/* Bytes of the packed weight buffer: N*K/4 for the two-bit sets, N*K/2 for INT4, 3*N*K/8 for INT3, after
 * padding N and the (two-bit) words per row to multiples of 16.  0 on bad input. */
size_t qift_packed_bytes(int N, int K, int levels);

/* Bytes of scratch qift_w2a4_linear / qift_w4a4_linear can use for this problem, rounded up to 1 KiB:
 *   M = 1                 0 (decode route);
 *   2 <= M <= 64          M*K + 512 when K is a whole number of 16-word slices (QIFT_ROUTE_DECODE_ROWS: the
 *                         activations re-laid out for a row-split kernel plus the token sums), else 0
 *                         for M <= 16 or 4*M above;
 *   64 < M <= 512         4*M (QIFT_ROUTE_PREFILL up to 128 rows, QIFT_ROUTE_PREFILL_FUSED_PAIR above:
 *                         the per-token sums of q_a);
 *   M > 512               N*K (QIFT_ROUTE_PREFILL_PAIR: the codes decoded to int8 once per call).
 * With less than this (or NULL) the call still runs when a route without scratch exists -- M <= 16
 * falls back to the K-split decode kernel, 17..64 rows to the fused prefill route if 4*M bytes were
 * passed -- and returns QIFT_ERR_WORKSPACE otherwise.  qift_workspace_bytes_route gives the figure
 * for an explicit route.
 * INT3 has two product routes besides the generic one: the row-split decode kernel for 1 <= M <= 16
 * (M*K + 512 bytes) and the decode-to-int8 GEMM routes above that (N*K bytes). */
size_t qift_workspace_bytes(int M, int N, int K, int levels);
size_t qift_workspace_bytes_route(int M, int N, int K, int levels, int route);

/* S1 (weight quantizer + packer).  Sec. 1 Eq. 1, Sec. 3.3, Sec. 3.5.
 *   W       in   fp32 [N,K], ALREADY rotated (this call never rotates)
 *   s_n     in for QIFT_SCALE_GIVEN (must be > 0), out otherwise; fp32 [N]
 *   packed  out  qift_packed_bytes(N,K,levels) bytes of uint32 words in the tiled order below
 * Code of a weight: t = w / s_n (IEEE division).  No-zero sets: nearest level, an exact midpoint
 * goes to the lower level, values beyond the outer levels saturate.  SYM / INT4: Eq. 1 literally,
 * round-half-to-even then clip to [-2,1] / [-8,7]; SYM stores q+2, INT4 stores q & 15.
 * Bits in a word: word j of a row holds codes k = 16j..16j+15; code k = 16j + 4t + b sits at bits
 * [8b+2t+1 : 8b+2t] (INT4: k = 8j + 4t + b at bits [8b+4t+3 : 8b+4t]), so (word >> 2t) & 0x03030303
 * is four consecutive-k codes, one per byte.
 * Order of the words in memory: tiles of 16 rows x 128 words (the last tile of a row block may be
 * narrower), row blocks outermost, then ascending k.  Inside a tile, 16-byte groups of four
 * consecutive words of one row, group index ((slice*2 + half)*32 + (row%8)*4 + quad) with
 * slice = (j%128)/16, half = (row%16)/8, quad = (j%16)/4.  Rows and words per row are padded to
 * multiples of 16 with zero words (no padding for any LLaMA shape).  A tile is one 8 KB contiguous
 * block, and the 32 groups a warp needs for one mma step are 512 contiguous bytes.
 * INT3 (q & 7 of Eq. 1 with b = 3, clip to [-4,3]) is stored as two planes, level = (c & 3) - 4 (c >> 2):
 * the two low bits of the codes in words exactly as above, and the third bit 32 to a word -- high word h of
 * a row covers low words 2h and 2h+1, and the bit of code k = 16j + 4t + b sits in byte b at position
 * 4 (j%2) + {0,2,1,3}[t], so that the bits of planes t and t+1 (t even) lie two positions apart: with the
 * even planes' activations multiplied by four both halves of a product instruction carry one place value.
 * The planes are interleaved slice by slice: a slice (16 low words of the 16 rows of a row block) is 1536
 * contiguous bytes, 1024 of low words in the group order above followed by 512 of high words (group
 * (row%8)*4 + quad: the two high words of rows row%8 and row%8 + 8), slices in ascending k inside a row
 * block of 24 * pitch words; any run of slices of a row block is therefore one contiguous piece.
 * Requires K % 16 == 0 (K % 8 == 0 for INT4, K % 32 == 0 for INT3) and K <= 16384. */
int qift_pack_weights(const float* W, int N, int K, int levels, int scale_mode, float* s_n,
                      uint32_t* packed, void* stream);

/* Inverse of the packed layout, for tests: codes uint8 [N,K] (INT4: the nibble 0..15; INT3: 0..7). */
int qift_unpack_codes(const uint32_t* packed, int N, int K, int levels, uint8_t* codes, void* stream);

/* S0 (offline rotation, Sec. 3.1 / Sec. 4.1): Y = X Q with Q = blockdiag(H_B) / sqrt(B), H_B the
 * Sylvester-Walsh matrix in natural order, applied to every row of X fp32 [M,K] along K.  fp32
 * butterfly with stages in ascending stride, then one multiply by (float)(1/sqrt(B)).
 * had_block B: a power of two >= 2 dividing K (block-diagonal Sylvester blocks), or B = K when K = 28 * 2^p
 * (p >= 4; e.g. 14336 = 28 * 512): the full-dimension rotation H_28 (x) H_{2^p} / sqrt(K), H_28 by Paley's
 * second construction (q = 13), the sum over the 28 blocks taken in ascending block order in fp32 -- there is
 * no Sylvester matrix of such an order and the block-diagonal form rotates only inside blocks of 2^p.
 * K <= 16384, K % 16 == 0.  In place (Y == X) is allowed. */
int qift_rotate(const float* X, int M, int K, int had_block, float* Y, void* stream);

/* S2 + S3 (online rotation + per-token symmetric INT4 quantizer; Eq. 1 with b = 4, Sec. 4.1).
 *   X        in  [M,K] fp32 or bf16 (bf16 is widened exactly)
 *   had_block    0 = no rotation, else as for qift_rotate (a power of two >= 2 dividing K, or K = 28 * 2^p)
 *   clip_ratio   the paper uses 0.9; must be in (0, 1]
 *   q_a      out int8 [M,K], one value of [-8,7] per byte
 *   s_a      out fp32 [M]
 * u = blockwise H x (unnormalised); s_u = (amax*clip)/7 (1 for a zero row);
 * q = clamp(rint(u / s_u), -8, 7); s_a = s_u * (float)(1/sqrt(B)).   K <= 16384, K % 16 == 0. */
int qift_quantize_act(const void* X, int x_dtype, int M, int K, int had_block, float clip_ratio,
                      int8_t* q_a, float* s_a, void* stream);

/* S4 + S5 (exact integer product, then the channel and token scales in the epilogue: Sec. 1;
 * Sec. 3.6 decoded small signed integer levels) for the two-bit sets MNZ, POT, SYM.
 *   packed, s_n   from qift_pack_weights
 *   q_a, s_a      from qift_quantize_act
 *   Y         out [M,N] fp32 or bf16 (round to nearest even): ((float)acc * s_a[m]) * s_n[n]
 *   acc_debug out int32 [M,N] accumulators, or NULL
 *   workspace     >= qift_workspace_bytes(M,N,K,levels) bytes, 256-byte aligned; may be NULL when 0
 * M <= 16 takes a decode route (the row-split one up to 64 rows when its scratch is passed), 16 < M <= 512 the
 * fused prefill routes, larger M the CTA-pair scratch route. */
int qift_w2a4_linear(const uint32_t* packed, const float* s_n, int levels, const int8_t* q_a,
                     const float* s_a, int M, int N, int K, void* Y, int y_dtype, int32_t* acc_debug,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Same for INT4 weights (the W4A4 layers of the layer-wise mixed-precision setting, Sec. 4.4). */
int qift_w4a4_linear(const uint32_t* packed, const float* s_n, const int8_t* q_a, const float* s_a,
                     int M, int N, int K, void* Y, int y_dtype, int32_t* acc_debug, void* workspace,
                     size_t workspace_bytes, void* stream);

/* Same for INT3 weights (W3A4, the three-bit point the mixed-precision stacks are compared with at equal
 * average bits: Sec. 4.4).  1 <= M <= 16 with the scratch of qift_workspace_bytes takes the row-split decode
 * kernel (two launches: activations re-laid out, then the product), larger M decodes the codes to int8
 * and runs the tensor-core GEMM (one CTA per tile up to 512 rows, CTA pairs above); without scratch the
 * generic kernel runs. */
int qift_w3a4_linear(const uint32_t* packed, const float* s_n, const int8_t* q_a, const float* s_a,
                     int M, int N, int K, void* Y, int y_dtype, int32_t* acc_debug, void* workspace,
                     size_t workspace_bytes, void* stream);

/* The calls above with the kernel route chosen by the caller (tests and benchmarks).
 * INT3 is served by QIFT_ROUTE_GENERIC, QIFT_ROUTE_DECODE_ROWS (here from M = 1, up to 16 rows),
 * QIFT_ROUTE_PREFILL_SCRATCH and QIFT_ROUTE_PREFILL_PAIR.
 * QIFT_ERR_UNSUPPORTED_SHAPE when the route cannot serve the shape. */
int qift_linear_route(const uint32_t* packed, const float* s_n, int levels, const int8_t* q_a,
                      const float* s_a, int M, int N, int K, void* Y, int y_dtype, int32_t* acc_debug,
                      void* workspace, size_t workspace_bytes, int route, void* stream);

/* Whole layer in one call, S2..S5: qift_quantize_act followed by the product, X and Y on the device.
 *   scratch  >= qift_forward_scratch_bytes(...) bytes of device memory, 256-byte aligned; holds
 *            q_a, s_a and (for M > 16) the prefill workspace.  Contents are undefined afterwards. */
size_t qift_forward_scratch_bytes(int M, int N, int K, int levels, int x_dtype, int y_dtype);
int qift_forward(const void* X, int x_dtype, int M, int K, int had_block, float clip_ratio,
                 const uint32_t* packed, const float* s_n, int levels, int N, void* Y, int y_dtype,
                 void* scratch, size_t scratch_bytes, void* stream);

/* The same with X and Y in HOST memory (pinned memory makes the copies asynchronous): the call
 * enqueues the host-to-device copy of X, the layer, and the device-to-host copy of Y on `stream`;
 * Y_host is valid once the stream has been synchronized.  The scratch additionally holds the
 * device copies of X and Y (qift_forward_scratch_bytes already counts them). */
int qift_forward_host(const void* X_host, int x_dtype, int M, int K, int had_block, float clip_ratio,
                      const uint32_t* packed, const float* s_n, int levels, int N, void* Y_host,
                      int y_dtype, void* scratch, size_t scratch_bytes, void* stream);

/* ---- Several products of ONE activation, weights decoded ahead of their use --------------------
 * (Sec. 3.1: the layer pipeline; the paper describes no kernels, so the scheduling is this library's.)
 * In a transformer layer q / k / v read the same activation, and so do gate / up: it needs rotating and
 * quantizing once.  qift_forward_multi runs S2 + S3 once on X and then S4 + S5 for every listed output.
 * With more than 128 token rows the products run as ONE launch of the CTA-pair tensor-core GEMM over the
 * channel tiles of all outputs, reading int8 levels decoded from the packed codes into `levels_buf`
 * (qift_levels_bytes; output i at the sum of the earlier outputs' N*K rounded up to 1 KiB each).
 *
 * Decoding ahead: the decoding of a product's codes needs nothing but the codes, so a call can do it for
 * the NEXT call while its own GEMM runs (extra warps of the GEMM kernel; the GEMM leaves most issue slots
 * free).  Pass in `ahead` the outputs (only packed and N are read), K and level set of the next call and
 * the buffer that call will pass as its levels_buf; the next call then passes levels_ready = 1 and skips its
 * own decoding pass.  A caller walking a layer stack alternates two levels buffers.  The first call of a
 * chain (levels_ready = 0) decodes its own codes before its GEMM, as qift_w2a4_linear does.
 * `ahead` is a list (`next`): a call may decode for several later calls, each into that call's own buffer, so that
 * a long product (gate / up, down) carries the decoding for the short ones (q / k / v, o) of the next layer as well;
 * the caller then keeps as many levels buffers as calls lie between a decoding and its use.
 *
 *   X            dev [M,K] fp32 or bf16;  had_block, clip_ratio as for qift_quantize_act
 *   outputs      HOST array of 1..4 outputs: packed / s_n from qift_pack_weights (all with this K and
 *                level set), Y dev [M,N] (fp32 or bf16 per y_dtype), acc_debug dev int32 [M,N] or NULL
 *   scratch      dev, >= qift_forward_multi_scratch_bytes(...), 256-byte aligned: q_a, s_a and (M <= 128)
 *                the workspace of the per-output routes; undefined afterwards
 *   levels_buf   dev, >= qift_levels_bytes(K, outputs, count), 256-byte aligned; needed when M > 128.
 *                levels_ready = 1 promises it already holds the decoded levels of exactly these outputs
 *                (written by the previous call's `ahead`); nothing can check that promise
 *   ahead        HOST, or NULL.  With M <= 128 the call still honours it (separate decoding launches).
 * Results are bit-identical to qift_quantize_act + qift_w2a4_linear / qift_w4a4_linear per output.
 * Errors: INVALID_ARG (null pointers, count outside 1..4, enums), UNSUPPORTED_SHAPE, ALIGNMENT,
 * WORKSPACE (scratch or a levels buffer missing or too small), CUDA. */
typedef struct qift_linear_output {
    const uint32_t* packed; /* dev, from qift_pack_weights            */
    const float* s_n;       /* dev [N]                                */
    void* Y;                /* dev [M,N]                              */
    int32_t* acc_debug;     /* dev [M,N] INT32 accumulators, or NULL  */
    int N;
    int reserved;
} qift_linear_output;
typedef struct qift_decode_ahead {
    const qift_linear_output* outputs; /* host; a later call's outputs (packed and N are read)  */
    int count, K, levels;
    int reserved;
    void* levels_buf;                  /* dev; that call's levels_buf                            */
    size_t levels_bytes;
    const struct qift_decode_ahead* next; /* host; another later call to decode for, or NULL (at most 8 outputs over
                                             the whole chain)                                    */
} qift_decode_ahead;
size_t qift_levels_bytes(int K, const qift_linear_output* outputs, int count);
size_t qift_forward_multi_scratch_bytes(int M, int K, int levels, const qift_linear_output* outputs, int count);
int qift_forward_multi(const void* X, int x_dtype, int M, int K, int had_block, float clip_ratio, int levels,
                       const qift_linear_output* outputs, int count, int y_dtype, void* scratch, size_t scratch_bytes,
                       void* levels_buf, size_t levels_bytes, int levels_ready, const qift_decode_ahead* ahead,
                       void* stream);
/* The product part alone (S4 + S5 for every output) on an activation that qift_quantize_act has already
 * quantized: q_a int8 [M,K], s_a fp32 [M].  workspace >= qift_linear_multi_workspace_bytes(...) bytes
 * (0 for M > 128; NULL allowed then), 256-byte aligned; everything else as for qift_forward_multi. */
size_t qift_linear_multi_workspace_bytes(int M, int K, int levels, const qift_linear_output* outputs, int count);
int qift_linear_multi(const int8_t* q_a, const float* s_a, int M, int K, int levels, const qift_linear_output* outputs,
                      int count, int y_dtype, void* workspace, size_t workspace_bytes, void* levels_buf,
                      size_t levels_bytes, int levels_ready, const qift_decode_ahead* ahead, void* stream);

/* ---- Grouped decode path -----------------------------------------------------------------------
 * One persistent launch serves a list of independent layer problems that share M (<= 128 token rows; INT3 <= 16),
 * the level set, the dtypes and the clip ratio -- e.g. all linear modules of one decode step.  A W2
 * matrix is only 1-15 MB, far too little for one launch to reach an HBM steady state; the grouped
 * kernel streams the whole list back to back.  (No counterpart in the paper: it describes no kernels.)
 *
 * qift_group_plan validates the list and writes a plan into caller memory: `plan_host` (host) and
 * `plan_dev` (device, 128-byte aligned: plans of 33 .. 128 rows keep one tensor map per problem in it), each
 * qift_group_plan_bytes(count) bytes; the device copy is enqueued on `stream`.  The plan holds the caller's pointers, so it stays valid while those buffers live;
 * plan_host must stay alive and unchanged while the plan is used.  The run calls enqueue
 *   qift_group_quantize_act : S2+S3 for every problem (one launch)  X -> q_a, s_a
 *   qift_group_linear       : S4+S5 for every problem (one launch per 256 problems)  q_a, s_a -> Y;
 *                             needs the q_a, s_a and token sums that qift_group_quantize_act left
 *                             in the problems' buffers and in plan_dev
 *   qift_group_forward      : both.
 * Problems must not alias each other's Y, nor each other's q_a / s_a with one exception: modules that
 * read the SAME activation (q/k/v; gate/up) may name the same X, q_a, s_a (same K and had_block); the
 * plan then quantizes that activation once and every such product reads it.  K % 256 == 0 (two-bit sets, INT3) or
 * K % 128 == 0 (INT4), K <= 16384.  INT3 plans take up to 16 token rows. */
typedef struct qift_group_problem {
    const void* X;          /* dev [M,K] fp32 or bf16                         */
    const uint32_t* packed; /* dev, from qift_pack_weights                    */
    const float* s_n;       /* dev [N]                                        */
    int8_t* q_a;            /* dev [M,K] scratch: quantized activations       */
    float* s_a;             /* dev [M]   scratch: token scales                */
    void* Y;                /* dev [M,N] output                               */
    int32_t* acc_debug;     /* dev [M,N] INT32 accumulators, or NULL          */
    int N, K;
    int had_block;          /* 0 = no rotation, else as for qift_rotate       */
    int reserved;
} qift_group_problem;

size_t qift_group_plan_bytes(int count);
int qift_group_plan(const qift_group_problem* problems /*host*/, int count, int M, int levels, int x_dtype,
                    int y_dtype, float clip_ratio, void* plan_host, void* plan_dev, size_t plan_bytes,
                    void* stream);
int qift_group_quantize_act(const void* plan_host, const void* plan_dev, void* stream);
int qift_group_linear(const void* plan_host, const void* plan_dev, void* stream);
int qift_group_forward(const void* plan_host, const void* plan_dev, void* stream);

/* qift_group_forward with the activations and the results in HOST memory.  The caller lays all X of
 * the plan out in one device arena and all Y in another (the plan's X / Y pointers point into them)
 * and keeps host mirrors of both (pinned memory makes the copies asynchronous).  The call enqueues
 * one host-to-device copy of the X arena, the two grouped launches, and one device-to-host copy of
 * the Y arena; y_host is valid once `stream` has been synchronized. */
int qift_group_forward_host(const void* plan_host, const void* plan_dev, const void* x_host, void* x_dev,
                            size_t x_bytes, const void* y_dev, void* y_host, size_t y_bytes, void* stream);

/* ---- Product without any allocation by anyone ------------------------------------------------
 * (No counterpart in the paper: this is a packaging variant of qift_w2a4_linear's prefill route.)
 *
 * Some callers cannot allocate device memory at the moment they need the layer: code running inside
 * a region where cudaMalloc is forbidden or would synchronize the device (a latency-critical serving
 * loop, a plugin whose host hands it fixed buffers and no allocator, a stream that is being
 * captured), or a process whose memory pool is owned by another framework and already fully
 * committed.  The prefill route needs N*K bytes of scratch for the decoded int8 levels; this entry
 * point takes that scratch from an array that is compiled into the library instead of from the
 * caller.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   qift_static_scratch_bytes()   capacity of the built-in array (16 MiB): problems need N*K <= it.
 *   qift_w2a4_linear_static(...)  same arguments and results as qift_w2a4_linear (any M >= 1, the
 *                                 two-bit level sets), minus the workspace; always takes the
 *                                 prefill route.  QIFT_ERR_TOO_LARGE when N*K exceeds the capacity.
 *
 * The array lives in every GPU context that loads the library, until the process exits.  The first
 * call on each device looks up the array's device address (one cudaGetSymbolAddress, with that device
 * current); make that first call before starting any stream capture.  All calls on a device share
 * the one array and it keeps the previous call's bytes: every byte the product reads is rewritten by
 * the call itself, so nothing needs clearing, but two calls that can overlap on the GPU (different
 * streams without an ordering between them) race on it -- serialize them. */
size_t qift_static_scratch_bytes(void);
int qift_w2a4_linear_static(const uint32_t* packed, const float* s_n, int levels, const int8_t* q_a,
                            const float* s_a, int M, int N, int K, void* Y, int y_dtype,
                            int32_t* acc_debug, void* stream);

/* Prefill with RESIDENT decoded weights.  The prefill product is compute-bound and a B200 has room to
 * keep, beside the packed codes that the decode path streams, the same weights decoded to one int8 level
 * per byte (4x the packed size for the two-bit sets): qift_expand_weights writes them once,
 * qift_expanded_linear is then the tensor-core product alone (S4 + S5 on CTA pairs), with no
 * per-call decoding pass and no scratch.
 *   levels_out / levels_in  dev int8 [N][K] row-major, 256-byte aligned, N*K bytes; level(code[n][k])
 *                           (MNZ in its odd-integer form -3..3, s_n being the half-scale)
 *   other arguments as for qift_w2a4_linear; any M >= 1 (meant for M of a few hundred and more)
 * The paper has no counterpart (it keeps no second copy of the weights); results are bit-identical to
 * qift_w2a4_linear / qift_w4a4_linear. */
int qift_expand_weights(const uint32_t* packed, int N, int K, int levels, int8_t* levels_out, void* stream);
int qift_expanded_linear(const int8_t* levels_in, const float* s_n, const int8_t* q_a, const float* s_a, int M, int N,
                         int K, void* Y, int y_dtype, int32_t* acc_debug, void* stream);

/* ---------------------------------------------------------------------------------------------------
 * KV4: the 4-bit key / value cache of the paper's W2A4/KV4 setting (Sec. 4.1: keys and values quantized
 * asymmetrically with a clipping ratio of 0.95) and the single-query decode attention that reads it.
 *
 * Cache layout (device memory, owned by the caller), head-major, T_cap even:
 *   key codes   uint8 [H][T_cap][D/2]   two neighbouring dimensions of a token per byte (even one low)
 *   value codes uint8 [H][T_cap/2][D]   two consecutive tokens of a dimension per byte (even one low)
 *   scale fp32  [H][T_cap]              step s of the (token, head) vector
 *   zero  fp32  [H][T_cap]              its integer zero-point z (0..15) as a float; value = s * (code - z)
 * (a byte is then one tensor-core operand register of the product it feeds).  D must be 128.
 *
 * qift_kv4_quantize: quantizes T new tokens and writes them to cache slots t0 .. t0+T-1 of a key cache
 * (layout = QIFT_KV_KEYS) or a value cache (QIFT_KV_VALUES; a slot's partner nibble is preserved).
 *   X        in  [T][H][D] fp32 or bf16 (the layout a projection produces), 16-byte aligned
 *   had_block    0 / 1: no rotation; else a power of two <= D: orthonormal blockwise Hadamard first
 *                (keys: rotate the query the same way, e.g. with qift_rotate)
 *   clip         clipping ratio in (0, 1]; the paper uses 0.95
 *   per vector: lo = clip * min(0, min x), hi = clip * max(0, max x), s = (hi - lo) / 15 (1 if hi == lo),
 *   z = rint(-lo / s), code = clamp(rint(x / s) + z, 0, 15); fp32, IEEE division, round half to even.
 *
 * qift_kv4_attention_decode: out[h] = sum_t softmax_t(q[h] . K[t] / sqrt(D)) V[t] over tokens 0 .. T-1 of
 * KV head h / (Hq / Hkv), K and V dequantized on the fly; fp32 arithmetic.
 *   q        in  [Hq][D] fp32, in the basis the keys were quantized in
 *   out      out [Hq][D] fp32
 *   Hq / Hkv     1 .. 8
 *   workspace    >= qift_kv4_attention_workspace_bytes(T, Hq, Hkv) bytes, 16-byte aligned: partial results
 *                of the token splits (two launches: partial attention per split, then the merge)
 * Errors: INVALID_ARG (null pointer, T <= 0, T > T_cap, clip outside (0,1], layout), UNSUPPORTED_SHAPE
 * (D != 128, odd T_cap, T_cap > 2^24 in the attention, more than 8 query heads per KV head, had_block), ALIGNMENT, WORKSPACE, CUDA. */
enum { QIFT_KV_KEYS = 0, QIFT_KV_VALUES = 1 };
int qift_kv4_quantize(const void* X, int x_dtype, int T, int H, int D, int had_block, float clip_ratio, int t0,
                      int T_cap, int layout, uint8_t* codes, float* scale, float* zero, void* stream);
size_t qift_kv4_attention_workspace_bytes(int T, int Hq, int Hkv);
int qift_kv4_attention_decode(const float* q, const uint8_t* k_codes, const float* k_scale, const float* k_zero,
                              const uint8_t* v_codes, const float* v_scale, const float* v_zero, int T, int T_cap,
                              int Hq, int Hkv, int D, float* out, void* workspace, size_t workspace_bytes,
                              void* stream);

/* Quantizer diagnostics (not on the inference path).  Sec. 3.3 (list of evaluated grids), Sec. 4.5.1
 * (bucket diagnostic), Sec. 4.5.2 (scale-invariant ratio scan).
 *
 * qift_diag_grid_quantize: nearest-level quantization of rotated weights onto s_n * grid for ANY four
 * float levels (Lloyd-Max, NF2, Far-MNZ, or a deployable set written as floats).
 *   W      in   fp32 [N,K] device, 16-byte aligned; K <= 16384
 *   grid   in   HOST, four ascending levels, grid[3] > 0
 *   s_n    in for QIFT_SCALE_GIVEN, out otherwise; fp32 [N] device.  ABSMAX: the row's absolute maximum
 *               lands on grid[3]; MSE: the packer's sweep of 80 clipping ratios 1.00 .. 0.21, least
 *               fp64 squared error, first index on ties (an all-zero row gets 1)
 *   codes  out  uint8 [N,K] device, one code 0..3 per weight (index into grid); may be NULL
 * Code of a weight: t = w / s_n (IEEE fp32 division); the number of fp32 midpoints
 * (grid[i] + grid[i+1]) / 2 that t exceeds, so an exact midpoint goes to the lower level.  For the
 * no-zero sets this is the rule of qift_pack_weights.
 *
 * qift_diag_bucket_stats: per level c < L, count[c] = weights with code c and sqerr[c] = the sum of
 * (w - s_n * values[c])^2 over them in fp64; the shares of Sec. 4.5.1 are these over their totals.
 *   codes  in   uint8 [N,K] device (qift_unpack_codes or qift_diag_grid_quantize), 4-byte aligned
 *   values in   HOST, L level values (the level table of the set, or the float grid); L = 4 or 16
 *   count  out  uint64 [L] device;  sqerr out fp64 [L] device (both overwritten)
 * K % 4 == 0.  The order of the fp64 additions is not fixed: sums repeat to about 1e-15 relative.
 *
 * qift_diag_ratio_scan: for each ratio r, NMSE(r) = min over beta > 0 of
 * sum_i (x_i - Q(x_i))^2 / sum_i x_i^2 with Q the nearest of beta * {-1, -r, +r, +1}, and the beta
 * that attains it.  The minimum is exact: the magnitudes are sorted, and for every split of the sorted
 * samples into inner and outer level the error is a parabola in beta whose constrained minimum is
 * closed-form; the least over all n + 1 splits is the answer (fp64).
 *   x      in   fp32 [n] device (pooled, normalized weights); 1 <= n <= 2^28
 *   ratios in   HOST, R values in (0, 1]; 1 <= R <= 65535
 *   beta, nmse  out fp64 [R] device
 *   workspace   >= qift_diag_ratio_scan_workspace_bytes(n, R) bytes, device, 256-byte aligned
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE (sizes outside the ranges above), ALIGNMENT, WORKSPACE, CUDA. */
int qift_diag_grid_quantize(const float* W, int N, int K, const float* grid, int scale_mode, float* s_n,
                            uint8_t* codes, void* stream);
int qift_diag_bucket_stats(const float* W, const uint8_t* codes, int N, int K, const float* s_n,
                           const float* values, int L, unsigned long long* count, double* sqerr, void* stream);
size_t qift_diag_ratio_scan_workspace_bytes(long long n, int R);
int qift_diag_ratio_scan(const float* x, long long n, const double* ratios, int R, double* beta, double* nmse,
                         void* workspace, size_t workspace_bytes, void* stream);

/* Synchronizes `stream`, then reads and clears the device status word in which a kernel records an
 * expired bounded wait.  QIFT_OK, QIFT_ERR_TIMEOUT or QIFT_ERR_CUDA.  `detail` (host, may be NULL)
 * receives the raw word: bits 0-7 the waiting site, the rest the block index. */
int qift_device_status(void* stream, uint32_t* detail);

/* Self-test of the bounded device-side waits (test-only; the paper has no counterpart).  Every wait of a
 * kernel on an mbarrier gives up after a wall-time bound (two seconds by default), records where in the
 * status word and lets the kernel end normally; a product call whose kernel gave up has still returned
 * QIFT_OK (everything is asynchronous) and leaves Y unwritten -- qift_device_status is how a caller learns
 * of it.  This entry makes such a wait run out on purpose, with a short bound and without any fault:
 *   which = 0   one CTA waits for an mbarrier phase that nobody completes; site byte 0x7e
 *   which = 1   the CTA-pair prefill GEMM on one 256 x 256 x 128 tile whose producers issue no loads (the
 *               operands are the library's built-in scratch and are never read): the wait for operands
 *               (site 32) and the waits for the accumulator (site 33) run out, all roles leave, tensor
 *               memory is freed
 *   limit_us    the bound, 1 .. 1 000 000 microseconds
 * Afterwards qift_device_status returns QIFT_ERR_TIMEOUT once, with the site in bits 0-7 of `detail`, and
 * QIFT_OK on the next call.  INVALID_ARG for other arguments. */
int qift_selftest_wait_timeout(int which, unsigned int limit_us, void* stream);

/* Measurement helpers (no counterpart in the paper; used by the benchmark to calibrate its roofline
 * denominators on the GPU it runs on; neither touches the quantized layer).
 *   qift_calib_hbm_read   streams `bytes` of device memory at `buf` through 128-bit loads, writes nothing
 *                         (`sink`, dev, may be NULL, is only there to keep the loads alive): the read-only
 *                         HBM ceiling.  Time it with events on `stream`.
 *   qift_calib_mma_i8     every SM pair issues kblocks x 4 tcgen05.mma kind::i8 (256 x 256 x 32 each) back to
 *                         back on operands resident in shared memory, no loads in the loop: the rate of the
 *                         tensor pipe itself under the power limit.  *ops (host, may be NULL) receives the
 *                         integer operations of the launch (2 per multiply-add).  1 <= kblocks <= 2^20. */
int qift_calib_hbm_read(const void* buf, size_t bytes, unsigned int* sink, void* stream);
int qift_calib_mma_i8(int kblocks, double* ops, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QIFT_H_ */

// Qift rotated W2A4 / W4A4 quantized linear layer -- CPU ORACLE.
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, single-threaded C++17
// restatement of what the paper's quantized linear layer computes, written for checking the CUDA
// library against.  It shares no code, header, table or constant generator with the CUDA path and
// neither includes the other.  Only tests, the smoke check and the CPU-baseline / reference legs of
// the benchmark may call it.  Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC.
//
// What each function follows (paper = "Qift: Shift-Friendly No-Zero W2 Post-Training Quantization
// for Rotated W2A4/KV4 LLM Inference"):
//   orc_level_value      Sec. 3.3 level-set list (SYM-INT, MNZ, PoT-MNZ) and Eq. 1 with b = 4;
//                        MNZ is held in its half-scale odd-integer form {-3,-1,+1,+3} (Sec. 3.3,
//                        the identity {-1.5,-.5,.5,1.5} s = {-3,-1,1,3} s/2).
//   orc_wht_blocks       Sec. 3.1 / Sec. 4.1 (the default, unlearned Hadamard rotation): Sylvester-Walsh matrix
//                        in natural order applied by the textbook in-place butterfly, stages in
//                        ascending stride, fp32.
//   orc_rotate_weights   the same rotation with the orthonormal factor 1/sqrt(B) (offline, weights).
//   orc_hadamard28, orc_wht_kron28   full-dimension rotation for K = 28 * 2^p (14336 = 28 * 512), which
//                        has no Sylvester matrix: H_28 (Paley's second construction, q = 13) Kronecker H_{2^p}.
//   orc_quantize_act     Eq. 1 with b = 4 on the rotated row, symmetric, clipping ratio as an
//                        argument (Sec. 4.1 uses 0.9), one scale per token row.
//   orc_weight_scale     Sec. 3.5 / Sec. 4.5.1: per-output-channel scale, either max-range or the
//                        least-squared-error one of a sweep over clipping ratios.
//   orc_assign_codes     Sec. 3.5: every weight goes to the nearest level times the scale; Eq. 1 for SYM-INT, INT4.
//   orc_pack / unpack    Sec. 3.3 (a code has two bits): 16 two-bit codes (8 nibbles) per 32-bit word,
//                        words stored in 16-row x 128-word tiles (layout comment at orc_pack).
//   INT3 (level set 4)   Sec. 4.4: the W3A4 configuration that the mixed-precision tables compare with at three
//                        bits per weight -- Eq. 1 with b = 3, levels -4..3, same per-channel scale rules;
//                        stored as a two-bit plane plus a one-bit plane (layout comment at orc_pack).
//   orc_int_matmul       Sec. 3.6 decoded small signed integer levels times integer activations.
//   orc_epilogue*        Sec. 1: the channel scale is applied after the integer product, in the epilogue.
//   orc_kv4_quantize     Sec. 4.1: the KV cache is quantized to four bits asymmetrically with a
//                        clipping ratio (0.95 there), keys and values alike; the paper gives no
//                        more, so the rest is the usual asymmetric integer quantizer: one
//                        (scale, zero-point) pair per token and head over the head dimension, the
//                        range [min(x,0), max(x,0)] shrunk by the clipping ratio, 16 levels.
//   orc_kv4_pack/unpack  two 4-bit codes per byte, even dimension in the low nibble (keys);
//   orc_kv4_pack_token_pairs  values: two consecutive tokens of a dimension per byte (layout is the build's).
//   orc_kv4_attention    single-query scaled dot-product attention over the dequantized cache (the
//                        decode step whose memory traffic Sec. 1 calls the bottleneck), in fp64.
//   orc_grid_*           Sec. 3.3 grid list: the same nearest-level quantizer for any four float levels
//                        (Lloyd-Max, NF2, Far-MNZ next to the deployable sets), scale as in orc_weight_scale.
//   orc_bucket_stats     Sec. 4.5.1: per assigned level, the share of weights and of squared error.
//   orc_ratio_scan       Sec. 4.5.2: NMSE(r) = min over a global scale beta of the error of
//                        beta * {-1,-r,+r,+1} on pooled samples, relative to their power.
//
// Parity pins for every function live in the CPU test-suite (closed forms, brute force, printed
// table values); none is "parity unpinned" except the numeric value of a forward output on the real
// models, which the paper never prints.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

enum Levels { LV_MNZ = 0, LV_POT = 1, LV_SYM = 2, LV_INT4 = 3, LV_INT3 = 4 };
enum ScaleMode { SC_GIVEN = 0, SC_ABSMAX = 1, SC_MSE = 2 };

constexpr int kNumCandidates = 80;  // clipping ratios 1.00, 0.99, ..., 0.21

// Decoded integer level of a stored code.  Two-bit sets are indexed in ascending level order.
int level_of(int lv, int code) {
    switch (lv) {
        case LV_MNZ: { const int t[4] = {-3, -1, +1, +3}; return t[code & 3]; }
        case LV_POT: { const int t[4] = {-4, -1, +1, +4}; return t[code & 3]; }
        case LV_SYM: { const int t[4] = {-2, -1, 0, +1}; return t[code & 3]; }
        case LV_INT3: {  // two's-complement three-bit field
            int c = code & 7;
            return c >= 4 ? c - 8 : c;
        }
        default: {  // INT4: two's-complement nibble
            int c = code & 15;
            return c >= 8 ? c - 16 : c;
        }
    }
}

// Largest positive level: the value a row's (clipped) absolute maximum is mapped onto.
float top_level(int lv) {
    switch (lv) {
        case LV_MNZ: return 3.0f;
        case LV_POT: return 4.0f;
        case LV_SYM: return 1.0f;
        case LV_INT3: return 3.0f;
        default: return 7.0f;
    }
}

int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

// Nearest-level code of one weight given its channel scale.
int code_of(int lv, float w, float s) {
    const float t = w / s;  // IEEE fp32 division
    if (lv == LV_MNZ) {     // decision thresholds are the midpoints -2, 0, +2; exact ties go down
        return (t > -2.0f) + (t > 0.0f) + (t > 2.0f);
    }
    if (lv == LV_POT) {     // midpoints -2.5, 0, +2.5
        return (t > -2.5f) + (t > 0.0f) + (t > 2.5f);
    }
    if (lv == LV_SYM) {     // Eq. 1, b = 2: round half to even, clip to [-2, 1]
        return clampi((int)std::rint(t), -2, 1) + 2;
    }
    if (lv == LV_INT3) {    // Eq. 1, b = 3: clip to [-4, 3]
        return clampi((int)std::rint(t), -4, 3) & 7;
    }
    return clampi((int)std::rint(t), -8, 7) & 15;  // Eq. 1, b = 4
}

float row_absmax(const float* w, int K) {
    float a = 0.0f;
    for (int k = 0; k < K; ++k) {
        const float v = std::fabs(w[k]);
        if (v > a) a = v;
    }
    return a;
}

float inv_sqrt_block(int B) { return (float)(1.0 / std::sqrt((double)B)); }

uint16_t bf16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);  // NaN stays NaN
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

}  // namespace

extern "C" {

int orc_level_value(int lv, int code) { return level_of(lv, code); }

int orc_num_candidates() { return kNumCandidates; }

// Clipping ratio of sweep candidate i.
float orc_candidate_ratio(int i) { return (float)(100 - i) / 100.0f; }

// In-place unnormalised Walsh-Hadamard transform of every contiguous block of B entries of a row
// of length K (B a power of two dividing K).  H H^T = B I.
void orc_wht_blocks(float* row, int K, int B) {
    for (int base = 0; base < K; base += B) {
        float* x = row + base;
        for (int h = 1; h < B; h <<= 1) {
            for (int i = 0; i < B; ++i) {
                if ((i & h) == 0) {
                    const float a = x[i];
                    const float b = x[i + h];
                    x[i] = a + b;
                    x[i + h] = a - b;
                }
            }
        }
    }
}

// Hadamard matrix of order 28 by Paley's second construction with q = 13 (13 = 1 mod 4): with chi the
// quadratic character mod 13 and C the symmetric conference matrix of order 14
//   C = [0 1^T; 1 Q],  Q[i][j] = chi(i - j),   C C^T = 13 I,
// H = [C + I, C - I; C - I, -C - I] has entries +-1, is symmetric and satisfies H H^T = 28 I.
// H: 28 x 28, row-major, entries +1 / -1.
void orc_hadamard28(int8_t* H) {
    int chi[13];
    for (int a = 0; a < 13; ++a) chi[a] = (a == 0) ? 0 : -1;
    for (int x = 1; x < 13; ++x) chi[(x * x) % 13] = 1;
    int C[14][14];
    for (int i = 0; i < 14; ++i)
        for (int j = 0; j < 14; ++j) {
            if (i == 0 || j == 0) C[i][j] = (i == j) ? 0 : 1;
            else C[i][j] = chi[((i - j) % 13 + 13) % 13];
        }
    for (int i = 0; i < 14; ++i)
        for (int j = 0; j < 14; ++j) {
            const int d = (i == j) ? 1 : 0;
            H[i * 28 + j] = (int8_t)(C[i][j] + d);
            H[i * 28 + j + 14] = (int8_t)(C[i][j] - d);
            H[(i + 14) * 28 + j] = (int8_t)(C[i][j] - d);
            H[(i + 14) * 28 + j + 14] = (int8_t)(-C[i][j] - d);
        }
}

// Full-dimension rotation of a row of length K = 28 * P (P a power of two), unnormalised: the Kronecker
// product H_28 (x) H_P, i.e. the Sylvester butterfly on every contiguous block of P entries, then H_28
// across the 28 blocks at every position i < P.  Each output of the second step is the signed sum of its
// 28 inputs taken in ascending block order in fp32 (first term +-x_0, then one add or subtract per
// block).  (H_28 (x) H_P)(H_28 (x) H_P)^T = K I, and the matrix is symmetric.
void orc_wht_kron28(float* row, int K) {
    const int P = K / 28;
    orc_wht_blocks(row, K, P);
    int8_t H[28 * 28];
    orc_hadamard28(H);
    float x[28], y[28];
    for (int i = 0; i < P; ++i) {
        for (int j = 0; j < 28; ++j) x[j] = row[(size_t)j * P + i];
        for (int r = 0; r < 28; ++r) {
            float acc = (H[r * 28] > 0) ? x[0] : -x[0];
            for (int j = 1; j < 28; ++j) acc = (H[r * 28 + j] > 0) ? acc + x[j] : acc - x[j];
            y[r] = acc;
        }
        for (int r = 0; r < 28; ++r) row[(size_t)r * P + i] = y[r];
    }
}

// The rotation selected by `B`: a power of two dividing K -> block-diagonal Sylvester blocks of B;
// B = K = 28 * 2^p -> the full-dimension Kronecker rotation above.
static void wht_select(float* row, int K, int B) {
    if ((B & (B - 1)) == 0) orc_wht_blocks(row, K, B);
    else orc_wht_kron28(row, K);
}

// W <- W Q with Q = blockdiag(H_B) / sqrt(B), applied to each row along K (H is symmetric).
void orc_rotate_weights(float* W, int N, int K, int B) {
    const float r = inv_sqrt_block(B);
    for (int n = 0; n < N; ++n) {
        float* row = W + (size_t)n * K;
        wht_select(row, K, B);
        for (int k = 0; k < K; ++k) row[k] = row[k] * r;
    }
}

void orc_bf16_to_f32(const uint16_t* in, float* out, long long n) {
    for (long long i = 0; i < n; ++i) {
        const uint32_t u = (uint32_t)in[i] << 16;
        std::memcpy(&out[i], &u, 4);
    }
}

void orc_f32_to_bf16(const float* in, uint16_t* out, long long n) {
    for (long long i = 0; i < n; ++i) out[i] = bf16_rne(in[i]);
}

// Rotate (B > 0) and quantize each activation row to the INT4 range.
//   u   = H_B-blocks applied to x                      (unnormalised)
//   s_u = (amax * clip) / 7          (1 if the row is all zero)
//   q   = clamp(rint(u / s_u), -8, 7)
//   s_a = s_u / sqrt(B)              (the orthonormal factor is folded into the scale)
// `scratch` holds one row (K floats).
void orc_quantize_act(const float* X, int M, int K, int B, float clip, int8_t* q, float* s_a,
                      float* scratch) {
    for (int m = 0; m < M; ++m) {
        for (int k = 0; k < K; ++k) scratch[k] = X[(size_t)m * K + k];
        if (B > 1) wht_select(scratch, K, B);
        const float amax = row_absmax(scratch, K);
        float s_u = 1.0f;
        if (amax != 0.0f) {
            const float clipped = amax * clip;
            s_u = clipped / 7.0f;
        }
        for (int k = 0; k < K; ++k) {
            const float t = scratch[k] / s_u;
            q[(size_t)m * K + k] = (int8_t)clampi((int)std::rint(t), -8, 7);
        }
        s_a[m] = (B > 1) ? s_u * inv_sqrt_block(B) : s_u;
    }
}

// Sum of squared reconstruction errors of one row at scale s, fp64, ascending k.
double orc_row_sqerr(const float* w, int K, int lv, float s) {
    double e = 0.0;
    for (int k = 0; k < K; ++k) {
        const int c = code_of(lv, w[k], s);
        const double d = (double)w[k] - (double)s * (double)level_of(lv, c);
        e += d * d;
    }
    return e;
}

// Per-output-channel scale.  mode 1: amax / top level.  mode 2: sweep of 80 clipping ratios,
// smallest squared error, first index on ties.  best_idx (may be null) receives the chosen
// candidate (0 for ABSMAX), errs (may be null, [N*80]) every candidate's error.
void orc_weight_scale(const float* W, int N, int K, int lv, int mode, float* s_n, int* best_idx,
                      double* errs) {
    const float g = top_level(lv);
    for (int n = 0; n < N; ++n) {
        const float* w = W + (size_t)n * K;
        const float amax = row_absmax(w, K);
        int best = 0;
        float s = 1.0f;
        if (amax != 0.0f) {
            if (mode == SC_ABSMAX) {
                s = amax / g;
            } else {
                double best_e = 0.0;
                for (int i = 0; i < kNumCandidates; ++i) {
                    const float p = orc_candidate_ratio(i);
                    const float clipped = p * amax;
                    const float si = clipped / g;
                    const double e = orc_row_sqerr(w, K, lv, si);
                    if (errs) errs[(size_t)n * kNumCandidates + i] = e;
                    if (i == 0 || e < best_e) {
                        best_e = e;
                        best = i;
                        s = si;
                    }
                }
            }
        } else if (errs) {
            for (int i = 0; i < kNumCandidates; ++i) errs[(size_t)n * kNumCandidates + i] = 0.0;
        }
        s_n[n] = s;
        if (best_idx) best_idx[n] = best;
    }
}

void orc_assign_codes(const float* W, int N, int K, int lv, const float* s_n, uint8_t* codes) {
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            codes[(size_t)n * K + k] = (uint8_t)code_of(lv, W[(size_t)n * K + k], s_n[n]);
}

// Packed layout.
// Bits inside a word: word j of row n holds codes k = per*j .. per*j + per-1;
//   two-bit sets: k = 16 j + 4 t + b  ->  bits [8 b + 2 t + 1 : 8 b + 2 t]
//   INT4:         k =  8 j + 4 t + b  ->  bits [8 b + 4 t + 3 : 8 b + 4 t]
// so that (word >> (bits * t)) masked per byte yields four consecutive-k codes, one per byte.
// Order of the words in memory: tiles of 16 rows x 128 words (the last tile of a row block may be
// narrower), row blocks outermost, tiles of one row block in ascending k.  Inside a tile the words
// go in groups of four (16 bytes): group index ((slice * 2 + half) * 32 + (row % 8) * 4 + quad),
// where slice = (j % 128) / 16, quad = (j % 16) / 4, half = (row % 16) / 8; word j % 4 inside the
// group.  Rows are padded to a multiple of 16 and the words of a row to a multiple of 16, with zero
// words.
static inline int pad16(int N) { return (N + 15) / 16 * 16; }

static size_t word_address(int n, int j, int words_per_row) {
    const int pitch = pad16(words_per_row);
    const int rb = n / 16, r = n % 16, half = r / 8, g = r % 8;
    const int c = j / 128, jj = j % 128;
    const size_t tile = (size_t)rb * 16 * pitch + (size_t)c * 16 * 128;
    const int slice = jj / 16, quad = (jj % 16) / 4, e = jj % 4;
    return tile + (size_t)(((slice * 2 + half) * 32 + g * 4 + quad) * 4 + e);
}

// Three-bit codes (INT3) are stored as two planes, interleaved slice by slice so that any run of slices of
// a row block is one contiguous piece of memory:
//   low plane:  the two low bits of every code, 16 per word, bit positions as for the two-bit sets;
//   high plane: the third bit, 32 per word.  High word h of a row covers low words 2h and 2h+1; the bit of
//               code k = 16 j + 4 t + b (low word j, plane t, byte b) sits in byte b at position
//               4 (j % 2) + {0, 2, 1, 3}[t].
// A slice is 16 low words (256 codes) of the 16 rows of a row block: 384 words = 256 low words in the
// group order of the two-bit layout (group (half * 32 + (row % 8) * 4 + quad), word j % 4 inside) followed
// by 128 high words in groups of four: group ((row % 8) * 4 + quad), quad = (j % 16) / 4, holds the two
// high words of that quad for row half 0 and then for row half 1 (word 2 * half + (j / 2) % 2 of the group).
// Row blocks outermost (24 * pitch words each, pitch = low words per row padded to 16), slices in
// ascending k.  K must be a multiple of 32.
static size_t int3_low_address(int n, int j, int pitch) {
    const int rb = n / 16, r = n % 16, half = r / 8, g = r % 8;
    const int slice = j / 16, quad = (j % 16) / 4, e = j % 4;
    return (size_t)rb * 24 * pitch + (size_t)slice * 384 + (size_t)((half * 32 + g * 4 + quad) * 4 + e);
}
static size_t int3_high_address(int n, int j, int pitch) {  // j: the LOW word index of the code
    const int rb = n / 16, r = n % 16, half = r / 8, g = r % 8;
    const int slice = j / 16, quad = (j % 16) / 4, pair = (j / 2) % 2;
    return (size_t)rb * 24 * pitch + (size_t)slice * 384 + 256 + (size_t)((g * 4 + quad) * 4 + 2 * half + pair);
}
static int int3_high_bit(int j, int t, int b) {
    const int order[4] = {0, 2, 1, 3};
    return 8 * b + 4 * (j % 2) + order[t];
}

long long orc_packed_words(int N, int K, int lv) {
    if (lv == LV_INT3) return (long long)pad16(N) * pad16(K / 16) * 3 / 2;
    const int per = (lv == LV_INT4) ? 8 : 16;
    return (long long)pad16(N) * pad16(K / per);
}

void orc_pack(const uint8_t* codes, int N, int K, int lv, uint32_t* packed) {
    const long long total = orc_packed_words(N, K, lv);
    for (long long i = 0; i < total; ++i) packed[i] = 0;
    if (lv == LV_INT3) {
        const int pitch = pad16(K / 16);
        for (int n = 0; n < N; ++n)
            for (int k = 0; k < K; ++k) {
                const int j = k / 16, t = (k % 16) / 4, b = k % 4;
                const uint32_t c = codes[(size_t)n * K + k] & 7u;
                packed[int3_low_address(n, j, pitch)] |= (c & 3u) << (8 * b + 2 * t);
                packed[int3_high_address(n, j, pitch)] |= (c >> 2) << int3_high_bit(j, t, b);
            }
        return;
    }
    const int per = (lv == LV_INT4) ? 8 : 16;
    const int bits = (lv == LV_INT4) ? 4 : 2;
    const int words = K / per;
    for (int n = 0; n < N; ++n) {
        for (int j = 0; j < words; ++j) {
            uint32_t w = 0;
            for (int r = 0; r < per; ++r) {
                const int t = r / 4, b = r % 4;
                const uint32_t c = codes[(size_t)n * K + (size_t)j * per + r] & ((1u << bits) - 1u);
                w |= c << (8 * b + bits * t);
            }
            packed[word_address(n, j, words)] = w;
        }
    }
}

void orc_unpack(const uint32_t* packed, int N, int K, int lv, uint8_t* codes) {
    if (lv == LV_INT3) {
        const int pitch = pad16(K / 16);
        for (int n = 0; n < N; ++n)
            for (int k = 0; k < K; ++k) {
                const int j = k / 16, t = (k % 16) / 4, b = k % 4;
                const uint32_t low = (packed[int3_low_address(n, j, pitch)] >> (8 * b + 2 * t)) & 3u;
                const uint32_t high = (packed[int3_high_address(n, j, pitch)] >> int3_high_bit(j, t, b)) & 1u;
                codes[(size_t)n * K + k] = (uint8_t)(low | (high << 2));
            }
        return;
    }
    const int per = (lv == LV_INT4) ? 8 : 16;
    const int bits = (lv == LV_INT4) ? 4 : 2;
    const int words = K / per;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            const int j = k / per, r = k % per, t = r / 4, b = r % 4;
            codes[(size_t)n * K + k] =
                (uint8_t)((packed[word_address(n, j, words)] >> (8 * b + bits * t)) & ((1u << bits) - 1u));
        }
}

// acc[m][n] = sum_k level(code[n][k]) * q_a[m][k]; plain triple loop, int32 with an int64 shadow.
// Returns the number of entries whose int32 and int64 sums differ (0 = no overflow anywhere).
long long orc_int_matmul(const uint8_t* codes, int lv, const int8_t* q, int M, int N, int K,
                         int32_t* acc) {
    long long bad = 0;
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            int32_t a32 = 0;
            int64_t a64 = 0;
            for (int k = 0; k < K; ++k) {
                const int L = level_of(lv, codes[(size_t)n * K + k]);
                const int qa = (int)q[(size_t)m * K + k];
                a32 += L * qa;
                a64 += (int64_t)L * (int64_t)qa;
            }
            if ((int64_t)a32 != a64) ++bad;
            acc[(size_t)m * N + n] = a32;
        }
    }
    return bad;
}

// y = ((float)acc * s_a[m]) * s_n[n]
void orc_epilogue(const int32_t* acc, const float* s_a, const float* s_n, int M, int N, float* y) {
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            const float t = (float)acc[(size_t)m * N + n] * s_a[m];
            y[(size_t)m * N + n] = t * s_n[n];
        }
}

void orc_epilogue_bf16(const int32_t* acc, const float* s_a, const float* s_n, int M, int N,
                       uint16_t* y) {
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            const float t = (float)acc[(size_t)m * N + n] * s_a[m];
            y[(size_t)m * N + n] = bf16_rne(t * s_n[n]);
        }
}

// ------------------------------------------------------------------------------------------------
// KV4: asymmetric 4-bit key / value cache
// ------------------------------------------------------------------------------------------------
// Quantize `rows` vectors of length D (one per token and head).  With B > 1 the vector is first
// rotated by the ORTHONORMAL blockwise Hadamard (butterfly, then one multiply by 1/sqrt(B)): queries
// carry no per-vector scale into which the factor could be folded.
//   lo = clip * min(0, min_d u),  hi = clip * max(0, max_d u)       (zero always inside the range)
//   s  = (hi - lo) / 15            (s = 1, z = 0 if hi == lo)
//   z  = rint(-lo / s)             (integer zero-point, 0..15, stored as a float)
//   c  = clamp(rint(u / s) + z, 0, 15),   dequantized value  s * (c - z)
// All in fp32 with IEEE division and round-half-even.  codes: one per byte.  scratch: D floats.
void orc_kv4_quantize(const float* X, long long rows, int D, int B, float clip, uint8_t* codes, float* scale,
                      float* zero, float* scratch) {
    for (long long r = 0; r < rows; ++r) {
        for (int d = 0; d < D; ++d) scratch[d] = X[(size_t)r * D + d];
        if (B > 1) {
            orc_wht_blocks(scratch, D, B);
            const float f = inv_sqrt_block(B);
            for (int d = 0; d < D; ++d) scratch[d] = scratch[d] * f;
        }
        float mn = 0.0f, mx = 0.0f;
        for (int d = 0; d < D; ++d) {
            if (scratch[d] < mn) mn = scratch[d];
            if (scratch[d] > mx) mx = scratch[d];
        }
        const float lo = mn * clip, hi = mx * clip;
        float s = 1.0f, z = 0.0f;
        if (hi != lo) {
            const float range = hi - lo;
            s = range / 15.0f;
            const float nlo = -lo;
            z = (float)std::rint(nlo / s);
        }
        for (int d = 0; d < D; ++d) {
            const float t = scratch[d] / s;
            const int c = (int)std::rint(t) + (int)z;
            codes[(size_t)r * D + d] = (uint8_t)clampi(c, 0, 15);
        }
        scale[r] = s;
        zero[r] = z;
    }
}

void orc_kv4_pack(const uint8_t* codes, long long rows, int D, uint8_t* bytes) {
    for (long long r = 0; r < rows; ++r)
        for (int i = 0; i < D / 2; ++i)
            bytes[(size_t)r * (D / 2) + i] =
                (uint8_t)(codes[(size_t)r * D + 2 * i] | (codes[(size_t)r * D + 2 * i + 1] << 4));
}

// Value-cache byte order: the codes of two CONSECUTIVE TOKENS of one head at the same dimension share a
// byte (even token in the low nibble).  codes: [T][D] of one head, T even; bytes: [T/2][D].
void orc_kv4_pack_token_pairs(const uint8_t* codes, long long T, int D, uint8_t* bytes) {
    for (long long i = 0; i < T / 2; ++i)
        for (int d = 0; d < D; ++d)
            bytes[(size_t)i * D + d] = (uint8_t)(codes[(size_t)(2 * i) * D + d] | (codes[(size_t)(2 * i + 1) * D + d] << 4));
}

void orc_kv4_unpack(const uint8_t* bytes, long long rows, int D, uint8_t* codes) {
    for (long long r = 0; r < rows; ++r)
        for (int i = 0; i < D / 2; ++i) {
            const uint8_t b = bytes[(size_t)r * (D / 2) + i];
            codes[(size_t)r * D + 2 * i] = b & 15;
            codes[(size_t)r * D + 2 * i + 1] = b >> 4;
        }
}

// out[h][:] = sum_t softmax_t( q[h] . Khat[kv(h)][t] / sqrt(D) ) * Vhat[kv(h)][t][:],  kv(h) = h / (Hq / Hkv),
// Khat = ks * (kc - kz), Vhat likewise, everything in fp64.  Codes: one per byte, [Hkv][T][D];
// scales and zero-points [Hkv][T].  scratch: T doubles.
void orc_kv4_attention(const float* q, const uint8_t* kc, const float* ks, const float* kz, const uint8_t* vc,
                       const float* vs, const float* vz, int T, int Hq, int Hkv, int D, double* out, double* scratch) {
    const int group = Hq / Hkv;
    const double inv = 1.0 / std::sqrt((double)D);
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / group;
        double m = -INFINITY;
        for (int t = 0; t < T; ++t) {
            const size_t row = (size_t)kv * T + t;
            double dot = 0.0;
            for (int d = 0; d < D; ++d)
                dot += (double)q[(size_t)h * D + d] * ((double)ks[row] * ((double)kc[row * D + d] - (double)kz[row]));
            scratch[t] = dot * inv;
            if (scratch[t] > m) m = scratch[t];
        }
        double den = 0.0;
        for (int d = 0; d < D; ++d) out[(size_t)h * D + d] = 0.0;
        for (int t = 0; t < T; ++t) {
            const size_t row = (size_t)kv * T + t;
            const double p = std::exp(scratch[t] - m);
            den += p;
            for (int d = 0; d < D; ++d)
                out[(size_t)h * D + d] += p * ((double)vs[row] * ((double)vc[row * D + d] - (double)vz[row]));
        }
        for (int d = 0; d < D; ++d) out[(size_t)h * D + d] /= den;
    }
}

// ---------------------------------------------------------------------------------------------------
// Quantizer diagnostics (Sec. 4.5.1, 4.5.2) on four-level float grids (Sec. 3.3).
// A grid is four ascending float levels g[0] < g[1] < g[2] < g[3], g[3] > 0.

// Nearest level of w / s: the number of midpoints (g[i] + g[i+1]) / 2 below t; a tie goes to the
// lower level.  The division and the midpoints are fp32.
int orc_grid_code(const float* g, float w, float s) {
    const float t = w / s;
    int c = 0;
    for (int i = 0; i < 3; ++i) c += (t > (g[i] + g[i + 1]) * 0.5f);
    return c;
}

void orc_grid_codes(const float* W, int N, int K, const float* g, const float* s_n, uint8_t* codes) {
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            codes[(size_t)n * K + k] = (uint8_t)orc_grid_code(g, W[(size_t)n * K + k], s_n[n]);
}

double orc_grid_row_sqerr(const float* w, int K, const float* g, float s) {
    double e = 0.0;
    for (int k = 0; k < K; ++k) {
        const double d = (double)w[k] - (double)s * (double)g[orc_grid_code(g, w[k], s)];
        e += d * d;
    }
    return e;
}

// Per-row scale of a float grid: the row's absolute maximum (times a clipping ratio) lands on the
// largest level g[3]; mode as in orc_weight_scale (1: ratio 1, 2: sweep of the same 80 ratios).
void orc_grid_scale(const float* W, int N, int K, const float* g, int mode, float* s_n, int* best_idx,
                    double* errs) {
    for (int n = 0; n < N; ++n) {
        const float* w = W + (size_t)n * K;
        const float amax = row_absmax(w, K);
        int best = 0;
        float s = 1.0f;
        double best_e = 0.0;
        if (amax != 0.0f) {
            const int cands = mode == SC_ABSMAX ? 1 : kNumCandidates;
            for (int i = 0; i < cands; ++i) {
                const float si = (orc_candidate_ratio(i) * amax) / g[3];
                const double e = orc_grid_row_sqerr(w, K, g, si);
                if (errs) errs[(size_t)n * kNumCandidates + i] = e;
                if (i == 0 || e < best_e) {
                    best_e = e;
                    best = i;
                    s = si;
                }
            }
        }
        s_n[n] = s;
        if (best_idx) best_idx[n] = best;
    }
}

// Bucket diagnostic: for each level index c < L, how many weights carry code c and the sum of
// their squared reconstruction errors (w - s_n * value[c])^2 in fp64.  Shares are these divided
// by their totals.
void orc_bucket_stats(const float* W, const uint8_t* codes, int N, int K, const float* s_n, const float* value,
                      int L, long long* count, double* sqerr) {
    for (int c = 0; c < L; ++c) {
        count[c] = 0;
        sqerr[c] = 0.0;
    }
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            const int c = codes[(size_t)n * K + k];
            const double d = (double)W[(size_t)n * K + k] - (double)s_n[n] * (double)value[c];
            count[c] += 1;
            sqerr[c] += d * d;
        }
}

// Ratio scan.  For each ratio r the exact minimum over beta > 0 of
//     f(beta) = sum_i (x_i - Q(x_i))^2,   Q = nearest of beta * {-1, -r, +r, +1},
// divided by sum_i x_i^2.  With a = |x| sorted ascending, the j smallest samples go to the inner
// level exactly when the decision threshold beta (1 + r) / 2 lies in [a_(j-1), a_j]; on that
// interval f is the parabola  S2 - 2 beta (r A_j + B_j) + beta^2 (r^2 j + n - j)  with A_j the sum
// of the j smallest a and B_j the sum of the others, so its minimum there is at the vertex clamped
// to the interval; the answer is the least of these n + 1 minima.  fp64 throughout.
void orc_ratio_scan(const float* x, long long n, const double* r, int R, double* beta, double* nmse) {
    std::vector<double> a((size_t)n);
    double S1 = 0.0, S2 = 0.0;
    for (long long i = 0; i < n; ++i) a[(size_t)i] = std::fabs((double)x[i]);
    std::sort(a.begin(), a.end());
    for (long long i = 0; i < n; ++i) {
        S1 += a[(size_t)i];
        S2 += a[(size_t)i] * a[(size_t)i];
    }
    for (int q = 0; q < R; ++q) {
        const double rr = r[q];
        double best_f = S2, best_b = 0.0, A = 0.0;
        for (long long j = 0; j <= n; ++j) {
            const double lin = rr * A + (S1 - A);
            const double quad = rr * rr * (double)j + (double)(n - j);
            const double lo = (j == 0 ? 0.0 : a[(size_t)j - 1]) * 2.0 / (1.0 + rr);
            double b = lin / quad;
            if (b < lo) b = lo;
            if (j < n) {
                const double hi = a[(size_t)j] * 2.0 / (1.0 + rr);
                if (b > hi) b = hi;
            }
            const double f = S2 - 2.0 * b * lin + b * b * quad;
            if (f < best_f) {
                best_f = f;
                best_b = b;
            }
            if (j < n) A += a[(size_t)j];
        }
        beta[q] = best_b;
        nmse[q] = S2 > 0.0 ? best_f / S2 : 0.0;
    }
}

}  // extern "C"

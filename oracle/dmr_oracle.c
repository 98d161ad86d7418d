/*
 * CPU oracle for the low-bit / routed decoder linear layers of Dynamic Mixed-Precision
 * Routing.  TEST INFRASTRUCTURE ONLY: nothing on the product path may call this file.
 * It shares no code, header, table or constant with the CUDA library.
 *
 * What the paper fixes (and this file follows):
 *   - Sec. 3 (Problem Formulation): one base model at several numerical precisions; a
 *     routing index r_t per step chooses which precision serves that step.
 *   - Sec. 5, "Experimental Models and Precision", and App. "Quantization Detail":
 *     the low-precision model is W4A16 weight-only quantization of every decoder Linear
 *     (activations stay 16 bit); the high-precision model is bf16.
 *   - Sec. 4.2, "KL-to-Classification Mapping": y_t = 1 means high precision is needed.
 * The paper gives no quantization arithmetic.  The reading taken here is plain
 * round-to-nearest asymmetric min/max quantization with an integer zero point, a bf16
 * scale per group of `g` consecutive input features, and codes computed against the
 * STORED (bf16-rounded) scale; the steps are listed above each function.
 *
 * Everything floating point is IEEE binary64, compiled with -ffp-contract=off so that no
 * fused multiply-add replaces a written multiply and add.
 *
 * Pinned by tests (closed forms, exact rational arithmetic, brute force, numpy BLAS):
 *   oracle_pack / oracle_unpack, oracle_quantize, oracle_dequantize, oracle_lowbit_linear,
 *   oracle_dense_linear, oracle_routed_linear, oracle_route_partition.
 * Parity with the paper's own AWQ/GPTQ checkpoints is unpinned: the paper prints no
 * weight, scale, code or layer output, and those checkpoints need calibration data.
 *
 * Layouts (all row-major, contiguous):
 *   W  [N][K] bf16 bit patterns (uint16), N = out features, K = in features
 *   X  [M][K] bf16 bit patterns,          M = tokens / concurrent agent steps
 *   qweight [N][K*bits/32] uint32: 4-bit code k of a row sits in word k/8 at bits 4*(k%8)..+3;
 *                                  8-bit code k sits in word k/4 at bits 8*(k%4)..+7;
 *                                  3-bit codes (the W3A16 variant of Sec. 5 / App. "Quantization Detail"): every 32
 *                                  codes take three words.  Code i of the block, i < 30, sits in word i/10 at bits
 *                                  3*(i%10)..+2 when i%10 < 5 and at bits 16+3*(i%10-5)..+2 otherwise (five codes in
 *                                  each half-word, bit 15 and bit 31 left over); bit b of code 30 is bit 15 of word b,
 *                                  bit b of code 31 is bit 31 of word b.  (The paper gives no 3-bit layout: its W3
 *                                  checkpoint is expanded to fp16 at load time.  This one is defined by this library.)
 *   scales  [N][K/g] bf16 bits,  zeros [N][K/g] uint8
 *   Y  [M][N] binary64
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 5

/* ---------- bf16 <-> binary64 ---------- */

/* bf16 is the top half of a binary32: widen exactly. */
static double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int bf16_is_finite(uint16_t b) { return (b & 0x7F80u) != 0x7F80u; }

/*
 * Nearest bf16 to a positive finite binary64, ties to even, as a bit pattern.
 * Works by searching the bf16 lattice directly instead of manipulating bit fields:
 * find the largest positive bf16 `lo` with value <= x, then choose between lo and lo+1
 * by exact comparison of the two distances (both differences are exact in binary64
 * because x, lo and lo+1 lie within a factor 2 of each other or the gap is a power of 2).
 * Returns 0 for x below half the smallest subnormal; 0x7F80 (infinity) if x rounds past
 * the largest finite bf16.
 */
static uint16_t f64_to_bf16_rne_pos(double x) {
    uint16_t lo = 0, hi = 0x7F7F; /* positive finite patterns are ordered like integers */
    if (x >= bf16_to_f64(hi)) {
        /* gap above the largest finite value equals the gap below it: 2^120 */
        double top = bf16_to_f64(hi);
        double gap = top - bf16_to_f64(0x7F7E);
        return (x - top < gap / 2) ? hi : 0x7F80;
    }
    while (hi - lo > 1) { /* invariant: value(lo) <= x < value(hi) */
        uint16_t mid = (uint16_t)((lo + hi) / 2);
        if (bf16_to_f64(mid) <= x) lo = mid; else hi = mid;
    }
    double dlo = x - bf16_to_f64(lo);
    double dhi = bf16_to_f64((uint16_t)(lo + 1)) - x;
    if (dlo < dhi) return lo;
    if (dlo > dhi) return (uint16_t)(lo + 1);
    return (lo & 1u) ? (uint16_t)(lo + 1) : lo; /* tie: even significand */
}

uint16_t oracle_f64_to_bf16_rne(double x) {
    if (x == 0.0) return 0;
    if (x < 0) return (uint16_t)(0x8000u | f64_to_bf16_rne_pos(-x));
    return f64_to_bf16_rne_pos(x);
}

double oracle_bf16_to_f64(uint16_t b) { return bf16_to_f64(b); }

/* ---------- packing ---------- */

static int format_ok(int K, int bits, int g) {
    if (bits != 3 && bits != 4 && bits != 8) return 0;
    if (K <= 0 || g <= 0 || K % g != 0) return 0;
    if (bits == 3 ? K % 32 != 0 : K % (32 / bits) != 0) return 0;
    return 1;
}

static int words_per_row(int K, int bits) { return bits == 3 ? K / 32 * 3 : K / (32 / bits); }

/* where code i (0..29) of a 32-code block of 3-bit codes sits: word index and shift */
static void w3_place(int i, int *word, int *shift) {
    *word = i / 10;
    int j = i % 10;
    *shift = j < 5 ? 3 * j : 16 + 3 * (j - 5);
}

/* code k of one packed row */
static uint32_t code_at(const uint32_t *row, int k, int bits) {
    if (bits == 3) {
        const uint32_t *w = row + (size_t)(k / 32) * 3;
        int i = k % 32;
        if (i < 30) {
            int word, shift;
            w3_place(i, &word, &shift);
            return (w[word] >> shift) & 7u;
        }
        int bit = i == 30 ? 15 : 31;
        return ((w[0] >> bit) & 1u) | (((w[1] >> bit) & 1u) << 1) | (((w[2] >> bit) & 1u) << 2);
    }
    int per = 32 / bits;
    return (row[k / per] >> (bits * (k % per))) & ((1u << bits) - 1u);
}

/* codes [N][K] uint8 (each < 2^bits) -> qweight [N][K*bits/32] */
int oracle_pack(const uint8_t *codes, int N, int K, int bits, uint32_t *qweight) {
    if (bits != 3 && bits != 4 && bits != 8) return ORACLE_ERR_ARG;
    if (bits == 3 ? K % 32 != 0 : K % (32 / bits) != 0) return ORACLE_ERR_ARG;
    int words = words_per_row(K, bits);
    for (int n = 0; n < N; ++n) {
        uint32_t *row = qweight + (size_t)n * words;
        for (int j = 0; j < words; ++j) row[j] = 0;
        for (int k = 0; k < K; ++k) {
            uint32_t c = codes[(size_t)n * K + k];
            if (bits == 3) {
                uint32_t *w = row + (size_t)(k / 32) * 3;
                int i = k % 32;
                if (i < 30) {
                    int word, shift;
                    w3_place(i, &word, &shift);
                    w[word] |= (c & 7u) << shift;
                } else {
                    int bit = i == 30 ? 15 : 31;
                    for (int b = 0; b < 3; ++b) w[b] |= ((c >> b) & 1u) << bit;
                }
            } else {
                int per = 32 / bits;
                row[k / per] |= (c & ((1u << bits) - 1u)) << (bits * (k % per));
            }
        }
    }
    return ORACLE_OK;
}

int oracle_unpack(const uint32_t *qweight, int N, int K, int bits, uint8_t *codes) {
    if (bits != 3 && bits != 4 && bits != 8) return ORACLE_ERR_ARG;
    if (bits == 3 ? K % 32 != 0 : K % (32 / bits) != 0) return ORACLE_ERR_ARG;
    int words = words_per_row(K, bits);
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) codes[(size_t)n * K + k] = (uint8_t)code_at(qweight + (size_t)n * words, k, bits);
    return ORACLE_OK;
}

/* ---------- quantization ---------- */

/*
 * One group of g weights -> (scale bits, zero, codes).  Steps, with qmax = 2^bits - 1:
 *   1. any NaN/Inf weight           -> error
 *   2. lo = min(0, min w), hi = max(0, max w)          (0 always representable)
 *   3. s64 = (hi - lo) / qmax;  all-zero group: s64 = 1
 *   4. s = nearest bf16 to s64 (ties to even); if s < 2^-126 (zero or subnormal) s = 2^-126
 *   5. z = clamp(rint(-lo / s), 0, qmax)               (rint: nearest, ties to even)
 *   6. q_k = clamp(rint(w_k / s) + z, 0, qmax)         (round first, then add integer z)
 */
static int quantize_group(const uint16_t *w, int g, int bits, uint16_t *scale_bits,
                          uint8_t *zero, uint8_t *codes) {
    double qmax = (double)((1 << bits) - 1);
    double lo = 0.0, hi = 0.0;
    for (int k = 0; k < g; ++k) {
        if (!bf16_is_finite(w[k])) return ORACLE_ERR_NONFINITE;
        double v = bf16_to_f64(w[k]);
        if (v < lo) lo = v;
        if (v > hi) hi = v;
    }
    double s64 = (hi == lo) ? 1.0 : (hi - lo) / qmax;
    uint16_t sb = oracle_f64_to_bf16_rne(s64);
    if (sb < 0x0080u) sb = 0x0080u; /* smallest normal bf16, 2^-126 */
    double s = bf16_to_f64(sb);
    double z = rint(-lo / s);
    if (z < 0.0) z = 0.0;
    if (z > qmax) z = qmax;
    for (int k = 0; k < g; ++k) {
        double q = rint(bf16_to_f64(w[k]) / s) + z;
        if (q < 0.0) q = 0.0;
        if (q > qmax) q = qmax;
        codes[k] = (uint8_t)q;
    }
    *scale_bits = sb;
    *zero = (uint8_t)z;
    return ORACLE_OK;
}

/* group == 0 means per-channel (one group spanning all of K). codes_out [N][K] may be NULL. */
int oracle_quantize(const uint16_t *W, int N, int K, int bits, int group,
                    uint32_t *qweight, uint16_t *scales, uint8_t *zeros, uint8_t *codes_out) {
    int g = group == 0 ? K : group;
    if (N <= 0 || !format_ok(K, bits, g)) return ORACLE_ERR_ARG;
    int G = K / g, words = words_per_row(K, bits);
    int err = ORACLE_OK;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        uint8_t *row = (uint8_t *)malloc((size_t)K);
        int row_err = ORACLE_OK;
        for (int j = 0; j < G; ++j) {
            int e = quantize_group(W + (size_t)n * K + (size_t)j * g, g, bits,
                                   &scales[(size_t)n * G + j], &zeros[(size_t)n * G + j],
                                   row + (size_t)j * g);
            if (e != ORACLE_OK) row_err = e;
        }
        if (row_err == ORACLE_OK) {
            oracle_pack(row, 1, K, bits, qweight + (size_t)n * words);
            if (codes_out) memcpy(codes_out + (size_t)n * K, row, (size_t)K);
        } else {
#pragma omp atomic write
            err = row_err;
        }
        free(row);
    }
    return err;
}

/* What[n][k] = s * (q - z) exactly (binary64); What_bf16 (optional) = nearest bf16 of it. */
int oracle_dequantize(const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                      int N, int K, int bits, int group, double *What, uint16_t *What_bf16) {
    int g = group == 0 ? K : group;
    if (N <= 0 || !format_ok(K, bits, g)) return ORACLE_ERR_ARG;
    int G = K / g, words = words_per_row(K, bits);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            uint32_t q = code_at(qweight + (size_t)n * words, k, bits);
            double s = bf16_to_f64(scales[(size_t)n * G + k / g]);
            double z = (double)zeros[(size_t)n * G + k / g];
            double v = s * ((double)q - z);
            if (What) What[(size_t)n * K + k] = v;
            if (What_bf16) What_bf16[(size_t)n * K + k] = oracle_f64_to_bf16_rne(v);
        }
    return ORACLE_OK;
}

/* ---------- linear layers ---------- */

/* one dequantized weight; rounded != 0 gives the nearest-bf16 version (diagnostic) */
static double dq_weight(const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                        int K, int bits, int g, int n, int k, int rounded) {
    int G = K / g, words = words_per_row(K, bits);
    uint32_t q = code_at(qweight + (size_t)n * words, k, bits);
    double s = bf16_to_f64(scales[(size_t)n * G + k / g]);
    double z = (double)zeros[(size_t)n * G + k / g];
    double v = s * ((double)q - z);
    return rounded ? bf16_to_f64(oracle_f64_to_bf16_rne(v)) : v;
}

static double lowbit_dot(const uint16_t *X, const uint32_t *qweight, const uint16_t *scales,
                         const uint8_t *zeros, int K, int bits, int g, int m, int n, int rounded) {
    double acc = 0.0;
    for (int k = 0; k < K; ++k)
        acc += bf16_to_f64(X[(size_t)m * K + k]) *
               dq_weight(qweight, scales, zeros, K, bits, g, n, k, rounded);
    return acc;
}

static double dense_dot(const uint16_t *X, const uint16_t *W, int K, int m, int n) {
    double acc = 0.0;
    for (int k = 0; k < K; ++k)
        acc += bf16_to_f64(X[(size_t)m * K + k]) * bf16_to_f64(W[(size_t)n * K + k]);
    return acc;
}

/* Y[m][n] = sum_k X[m][k] * What[n][k], k ascending. */
int oracle_lowbit_linear(const uint16_t *X, int M, const uint32_t *qweight, const uint16_t *scales,
                         const uint8_t *zeros, int N, int K, int bits, int group, int rounded,
                         double *Y) {
    int g = group == 0 ? K : group;
    if (M < 0 || N <= 0 || !format_ok(K, bits, g)) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m)
            Y[(size_t)m * N + n] = lowbit_dot(X, qweight, scales, zeros, K, bits, g, m, n, rounded);
    return ORACLE_OK;
}

/* Y[m][n] = sum_k X[m][k] * W[n][k], k ascending. */
int oracle_dense_linear(const uint16_t *X, int M, const uint16_t *W, int N, int K, double *Y) {
    if (M < 0 || N <= 0 || K <= 0) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m)
            Y[(size_t)m * N + n] = dense_dot(X, W, K, m, n);
    return ORACLE_OK;
}

/* Row m uses the bf16 weights when mask[m] != 0 (high precision needed), else the low-bit ones. */
int oracle_routed_linear(const uint16_t *X, int M, const uint8_t *mask, const uint16_t *W,
                         const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                         int N, int K, int bits, int group, double *Y) {
    int g = group == 0 ? K : group;
    if (M < 0 || N <= 0 || !format_ok(K, bits, g)) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int m = 0; m < M; ++m)
            Y[(size_t)m * N + n] = mask[m] ? dense_dot(X, W, K, m, n)
                                           : lowbit_dot(X, qweight, scales, zeros, K, bits, g, m, n, 0);
    return ORACLE_OK;
}

/* Sampled outputs: out[i] = routed/low-bit/dense value at (ms[i], ns[i]).
 * mask == NULL: all rows low-bit if qweight != NULL, else all rows dense. */
int oracle_sampled_linear(const uint16_t *X, int M, const uint8_t *mask, const uint16_t *W,
                          const uint32_t *qweight, const uint16_t *scales, const uint8_t *zeros,
                          int N, int K, int bits, int group, int rounded,
                          const int32_t *ms, const int32_t *ns, int count, double *out) {
    int g = group == 0 ? K : group;
    if (qweight && !format_ok(K, bits, g)) return ORACLE_ERR_ARG;
    for (int i = 0; i < count; ++i)
        if (ms[i] < 0 || ms[i] >= M || ns[i] < 0 || ns[i] >= N) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < count; ++i) {
        int high = mask ? (mask[ms[i]] != 0) : (qweight == NULL);
        out[i] = high ? dense_dot(X, W, K, ms[i], ns[i])
                      : lowbit_dot(X, qweight, scales, zeros, K, bits, g, ms[i], ns[i], rounded);
    }
    return ORACLE_OK;
}

/* Stable partition of step indices by mask: idx_high lists m with mask[m] != 0 in ascending
 * order, idx_low the others in ascending order. */
int oracle_route_partition(const uint8_t *mask, int M, int32_t *idx_high, int32_t *idx_low,
                           int32_t *n_high, int32_t *n_low) {
    int h = 0, l = 0;
    for (int m = 0; m < M; ++m) {
        if (mask[m]) idx_high[h++] = m; else idx_low[l++] = m;
    }
    *n_high = h;
    *n_low = l;
    return ORACLE_OK;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

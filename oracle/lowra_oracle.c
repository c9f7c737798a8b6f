/*
 * CPU oracle for the LowRA quantized-LoRA linear-layer hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, scalar C written from the paper's description:
 * it is the definition that the CUDA library is checked against and the CPU baseline that the
 * benchmark times.  It shares no code, header, table or helper with the CUDA path, and the
 * product never calls it.
 *
 * What follows the paper, passage by passage:
 *   absmax / normalise : Section 4.1 "Groupwise Normalization" (64-element blocks scaled by the
 *                        block's maximum magnitude) and Appendix A.1 (the quantize kernel loads a
 *                        block, computes its maximum magnitude, stores it, normalises with it).
 *   bucket             : Section 4.1 "Per-Output-Channel Thresholds and Mappings" (thresholds are
 *                        the bin edges that turn a normalised value into a bitstring) and
 *                        Appendix A.1 (per-channel precision `Precs`, per-channel decision
 *                        boundaries).
 *   pack / layout      : Appendix A.1 (packed results written at the channel's offset) with the
 *                        precision-grouped row order of the build's problem statement.
 *   decode             : Appendix A.2 (unpack 1/2/4 bits, per-channel lookup table, multiply by
 *                        the block's absmax, write the output tensor).
 *   Lloyd-Max          : Section 5 (weights = block absmax, initial tables of Appendix F,
 *                        centroid update then midpoint thresholds) and Appendix G (E-step, M-step).
 *
 * Readings taken where the paper is silent (all listed in the design notes of the repository):
 * reciprocal-then-multiply normalisation in fp32, zero block -> normalised value 0, tie at a
 * threshold -> upper bucket, LSB-first bit order, classes ordered 1,2,4 bits with a stable
 * permutation, fp32 product rounded to bf16 with round-to-nearest-even.
 *
 * Pinned by tests/test_oracle_*.py: printed constants of Appendix F, brute force on 8x8
 * matrices, closed forms (1-bit sign quantiser), packed-size and round-trip invariants,
 * non-increasing Lloyd-Max distortion, exact recovery of 2^b-point data.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define TABLE_STRIDE 16 /* fp32 entries per row in the mapping / threshold tables */

/* ------------------------------------------------------------------------------------------ */
/* small helpers                                                                              */
/* ------------------------------------------------------------------------------------------ */
static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* fp32 -> bf16, round to nearest even; NaN stays a quiet NaN. */
static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u = f32_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static int class_of_bits(int b) { return b == 1 ? 0 : b == 2 ? 1 : b == 4 ? 2 : -1; }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

void oracle_f32_to_bf16(const float* x, uint16_t* out, int64_t n) {
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(x[i]);
}

/* ------------------------------------------------------------------------------------------ */
/* O1 absmax: a[r, g] = max over the G consecutive k of |W[r, k]| (natural row order)         */
/* ------------------------------------------------------------------------------------------ */
void oracle_absmax(const float* W, int64_t N, int64_t K, int64_t G, float* a /*[N, K/G]*/) {
    const int64_t nb = K / G;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r)
        for (int64_t g = 0; g < nb; ++g) {
            float m = 0.0f;
            for (int64_t k = g * G; k < (g + 1) * G; ++k) {
                float v = fabsf(W[r * K + k]);
                if (v > m) m = v;
            }
            a[r * nb + g] = m;
        }
}

/* O2 normalise: n = x * fl(1/a); n = 0 when a == 0. Two separately rounded fp32 operations. */
static float normalise(float x, float a) {
    if (a == 0.0f) return 0.0f;
    volatile float inv = 1.0f / a; /* volatile: keep the reciprocal a rounded fp32 value */
    volatile float n = x * inv;
    return n;
}

void oracle_normalise(const float* W, int64_t N, int64_t K, int64_t G, float* out /*[N,K]*/) {
    const int64_t nb = K / G;
    float* a = (float*)malloc(sizeof(float) * (size_t)(N * nb));
    oracle_absmax(W, N, K, G, a);
    for (int64_t r = 0; r < N; ++r)
        for (int64_t k = 0; k < K; ++k) out[r * K + k] = normalise(W[r * K + k], a[r * nb + k / G]);
    free(a);
}

/* O3 bucket: number of valid thresholds t_j (j < 2^b - 1) with t_j <= n; linear scan.
 * A value equal to a threshold therefore falls in the upper bucket. */
static int bucket(float n, const float* thr, int b) {
    int code = 0;
    const int nt = (1 << b) - 1;
    for (int j = 0; j < nt; ++j)
        if (thr[j] <= n) ++code;
    return code;
}

/* ------------------------------------------------------------------------------------------ */
/* O4 layout: classes ordered 1, 2, 4 bits; inside a class ascending original row index.      */
/* Returns 0, or -1 if a precision is not in {1,2,4}.                                         */
/* ------------------------------------------------------------------------------------------ */
int oracle_plan(const uint8_t* precs, int64_t N, int64_t K, int32_t* perm, int32_t* inv_perm,
                int32_t counts[3], uint64_t seg_off[3], uint64_t* packed_bytes) {
    static const int bits[3] = {1, 2, 4};
    int64_t p = 0;
    uint64_t off = 0;
    for (int c = 0; c < 3; ++c) {
        counts[c] = 0;
        seg_off[c] = off;
        for (int64_t r = 0; r < N; ++r) {
            if (class_of_bits(precs[r]) < 0) return -1;
            if (precs[r] == bits[c]) {
                perm[p] = (int32_t)r;
                inv_perm[r] = (int32_t)p;
                ++p;
                ++counts[c];
            }
        }
        off += (uint64_t)counts[c] * (uint64_t)K * (uint64_t)bits[c] / 8u;
    }
    *packed_bytes = off;
    return p == N ? 0 : -1;
}

/* Byte address of stored row p (given its class c and its rank q inside the class). */
static uint64_t row_offset(const uint64_t seg_off[3], int c, int64_t q, int64_t K, int b) {
    return seg_off[c] + (uint64_t)q * (uint64_t)K * (uint64_t)b / 8u;
}

/* ------------------------------------------------------------------------------------------ */
/* encode = O1 + O2 + O3 + O4                                                                 */
/* W [N,K] fp32 natural order; thresholds [N,16] natural order (first 2^b-1 valid);           */
/* packed [packed_bytes]; absmax [N, K/G] in STORED row order.                                */
/* codes_out (optional, may be NULL): [N,K] uint8 codes in natural row order.                 */
/* ------------------------------------------------------------------------------------------ */
int oracle_encode(const float* W, int64_t N, int64_t K, int64_t G, const uint8_t* precs,
                  const float* thresholds, uint8_t* packed, float* absmax, uint8_t* codes_out) {
    if (K % G != 0 || K % 8 != 0) return -2;
    int32_t* perm = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    int32_t* inv = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    int32_t counts[3];
    uint64_t seg_off[3], total;
    int rc = oracle_plan(precs, N, K, perm, inv, counts, seg_off, &total);
    if (rc != 0) { free(perm); free(inv); return rc; }
    memset(packed, 0, (size_t)total);
    const int64_t nb = K / G;
    const int64_t class_start[3] = {0, counts[0], (int64_t)counts[0] + counts[1]};
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < N; ++p) {
        const int64_t r = perm[p];
        const int b = precs[r];
        const int c = class_of_bits(b);
        uint8_t* row = packed + row_offset(seg_off, c, p - class_start[c], K, b);
        for (int64_t g = 0; g < nb; ++g) {
            float a = 0.0f;
            for (int64_t k = g * G; k < (g + 1) * G; ++k) {
                float v = fabsf(W[r * K + k]);
                if (v > a) a = v;
            }
            absmax[p * nb + g] = a;
            for (int64_t k = g * G; k < (g + 1) * G; ++k) {
                const float n = normalise(W[r * K + k], a);
                const int code = bucket(n, thresholds + r * TABLE_STRIDE, b);
                if (codes_out) codes_out[r * K + k] = (uint8_t)code;
                /* element k occupies bits [k*b, k*b+b) of the row's bitstream, LSB first */
                for (int i = 0; i < b; ++i) {
                    const int64_t bit = k * b + i;
                    if ((code >> i) & 1) row[bit >> 3] |= (uint8_t)(1u << (bit & 7));
                }
            }
        }
    }
    free(perm);
    free(inv);
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* O5 decode: out[perm[p], k] = bf16_rne( maps[perm[p], code] * absmax[p, k/G] )              */
/* maps [N,16] natural order; out [N,K] bf16 bit patterns, natural row order.                 */
/* ------------------------------------------------------------------------------------------ */
int oracle_decode(const uint8_t* packed, const float* absmax, const float* maps,
                  const uint8_t* precs, int64_t N, int64_t K, int64_t G, uint16_t* out) {
    if (K % G != 0 || K % 8 != 0) return -2;
    int32_t* perm = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    int32_t* inv = (int32_t*)malloc(sizeof(int32_t) * (size_t)N);
    int32_t counts[3];
    uint64_t seg_off[3], total;
    int rc = oracle_plan(precs, N, K, perm, inv, counts, seg_off, &total);
    if (rc != 0) { free(perm); free(inv); return rc; }
    const int64_t nb = K / G;
    const int64_t class_start[3] = {0, counts[0], (int64_t)counts[0] + counts[1]};
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < N; ++p) {
        const int64_t r = perm[p];
        const int b = precs[r];
        const int c = class_of_bits(b);
        const uint8_t* row = packed + row_offset(seg_off, c, p - class_start[c], K, b);
        for (int64_t k = 0; k < K; ++k) {
            int code = 0;
            for (int i = 0; i < b; ++i) {
                const int64_t bit = k * b + i;
                code |= ((row[bit >> 3] >> (bit & 7)) & 1) << i;
            }
            volatile float v = maps[r * TABLE_STRIDE + code] * absmax[p * nb + k / G];
            out[r * K + k] = f32_to_bf16_rne(v);
        }
    }
    free(perm);
    free(inv);
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* O7 weighted Lloyd-Max per row (Section 5, Appendices F and G)                              */
/* ------------------------------------------------------------------------------------------ */
/* Initial tables as printed in Appendix F. */
static const double INIT_MAP4[16] = {-1.0, -0.6961928, -0.5250731, -0.3949175, -0.28444138,
                                     -0.18477343, -0.09105, 0.0, 0.0795803, 0.1609302,
                                     0.2461123, 0.33791524, 0.44070983, 0.562617, 0.72295684, 1.0};
static const double INIT_MAP2[4] = {-1.0, 0.0, 0.3379, 1.0};
static const double INIT_THR2[3] = {-0.5, 0.16895762, 0.66895762};
static const double INIT_MAP1[2] = {-1.0, 1.0};
static const double INIT_THR1[1] = {0.0};

/* Copies the initial levels / thresholds for precision b (thresholds for 4 bits: midpoints of
 * consecutive printed levels, the listing gives none). */
void oracle_initial_tables(int b, double* maps /*[2^b]*/, double* thr /*[2^b-1]*/) {
    if (b == 1) { memcpy(maps, INIT_MAP1, sizeof INIT_MAP1); memcpy(thr, INIT_THR1, sizeof INIT_THR1); }
    else if (b == 2) { memcpy(maps, INIT_MAP2, sizeof INIT_MAP2); memcpy(thr, INIT_THR2, sizeof INIT_THR2); }
    else {
        memcpy(maps, INIT_MAP4, sizeof INIT_MAP4);
        for (int j = 0; j < 15; ++j) thr[j] = (INIT_MAP4[j] + INIT_MAP4[j + 1]) * 0.5;
    }
}

static int bucket64(double n, const double* thr, int nt) {
    int code = 0;
    for (int j = 0; j < nt; ++j)
        if (thr[j] <= n) ++code;
    return code;
}

static double distortion(const double* x, const double* w, const int* c, const double* y, int64_t n) {
    double d = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const double e = x[i] - y[c[i]];
        d += w[i] * e * e;
    }
    return d;
}

/* One row: x[i] normalised data, w[i] weights (block absmax); T iterations of
 *   E: assign by current thresholds (rule O3)
 *   M: y_j <- sum w x / sum w over bucket j (empty bucket keeps y_j)
 *   T: t_j <- (y_j + y_{j+1}) / 2
 * trace (optional) receives 2T values: the weighted distortion after every E and every M step. */
void oracle_lloyd_max_row(const double* x, const double* w, int64_t n, int b, int T,
                          double* y /*[2^b] in/out*/, double* t /*[2^b-1] in/out*/, double* trace) {
    const int L = 1 << b;
    int* c = (int*)malloc(sizeof(int) * (size_t)n);
    for (int it = 0; it < T; ++it) {
        for (int64_t i = 0; i < n; ++i) c[i] = bucket64(x[i], t, L - 1);
        if (trace) trace[2 * it] = distortion(x, w, c, y, n);
        double num[16], den[16];
        for (int j = 0; j < L; ++j) num[j] = den[j] = 0.0;
        for (int64_t i = 0; i < n; ++i) { num[c[i]] += w[i] * x[i]; den[c[i]] += w[i]; }
        for (int j = 0; j < L; ++j)
            if (den[j] > 0.0) y[j] = num[j] / den[j];
        if (trace) trace[2 * it + 1] = distortion(x, w, c, y, n);
        for (int j = 0; j + 1 < L; ++j) t[j] = (y[j] + y[j + 1]) * 0.5;
    }
    free(c);
}

/* Whole matrix: per row, learn only the assigned precision.  Output tables [N,16] fp32:
 * maps32 = (float)y, thr32[j] = (float)(((double)maps32[j] + (double)maps32[j+1]) / 2);
 * unused maps = 0, unused thresholds = +inf.  trace (optional): [N, 2T]. */
int oracle_lloyd_max(const float* W, int64_t N, int64_t K, int64_t G, const uint8_t* precs, int T,
                     float* maps, float* thresholds, double* trace) {
    if (K % G != 0) return -2;
    const int64_t nb = K / G;
    int bad = 0;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t r = 0; r < N; ++r) {
        const int b = precs[r];
        if (class_of_bits(b) < 0) { bad = 1; continue; }
        double* x = (double*)malloc(sizeof(double) * (size_t)K);
        double* w = (double*)malloc(sizeof(double) * (size_t)K);
        for (int64_t g = 0; g < nb; ++g) {
            float a = 0.0f;
            for (int64_t k = g * G; k < (g + 1) * G; ++k) {
                float v = fabsf(W[r * K + k]);
                if (v > a) a = v;
            }
            for (int64_t k = g * G; k < (g + 1) * G; ++k) {
                x[k] = (double)normalise(W[r * K + k], a);
                w[k] = (double)a;
            }
        }
        double y[16], t[15];
        oracle_initial_tables(b, y, t);
        oracle_lloyd_max_row(x, w, K, b, T, y, t, trace ? trace + r * 2 * T : NULL);
        const int L = 1 << b;
        float* m32 = maps + r * TABLE_STRIDE;
        float* t32 = thresholds + r * TABLE_STRIDE;
        for (int j = 0; j < TABLE_STRIDE; ++j) { m32[j] = 0.0f; t32[j] = INFINITY; }
        for (int j = 0; j < L; ++j) m32[j] = (float)y[j];
        for (int j = 0; j + 1 < L; ++j) t32[j] = (float)(((double)m32[j] + (double)m32[j + 1]) * 0.5);
        free(x);
        free(w);
    }
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------------------------------ */
/* O6, definition written out: C[m,n] = sum_k A[m,k] * B[k,n] in long double, row-major.      */
/* Only for pinning the library matmul used by the Python side on small cases.                */
/* ------------------------------------------------------------------------------------------ */
void oracle_matmul_naive(const double* A, const double* B, double* C, int64_t M, int64_t Kd, int64_t Nn) {
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < Nn; ++n) {
            long double acc = 0.0L;
            for (int64_t k = 0; k < Kd; ++k) acc += (long double)A[m * Kd + k] * (long double)B[k * Nn + n];
            C[m * Nn + n] = (double)acc;
        }
}

/* unused-symbol guard for bits_f32 */
float oracle_bits_to_f32(uint32_t u) { return bits_f32(u); }

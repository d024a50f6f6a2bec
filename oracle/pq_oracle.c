/*
 * pq_oracle.c -- plain CPU oracle for the PermuQuant per-group quantized linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
 * CUDA library must compute.  It shares no code, header, table or constant with the CUDA path
 * and must never be reached from the product path; only the test-suite, the smoke check and
 * the benchmark's CPU-baseline leg may load it.
 *
 * Arithmetic conventions (all IEEE-754, round-to-nearest-even, denormals kept; compiled with
 * -ffp-contract=off so a fused multiply-add happens only where fmaf() is written):
 *   - bf16 -> fp32 widening is exact.
 *   - Integer per-group quantization follows the paper's Eq. 1 (scale = group absmax / Q) and
 *     Eq. 2 (round, clip to [-Q, Q], multiply back), with Q = 2^(b-1) - 1 and round = half-to-even.
 *   - NVFP4 (the paper names the format in Sec. 4.4 but does not define it): E2M1 codes on
 *     {0, .5, 1, 1.5, 2, 3, 4, 6}, groups of 16 channels, one unsigned E4M3 scale per group
 *     (group absmax / 6 expressed in units of the tensor scale), one fp32 tensor scale.
 *   - Channel second moments (Assumption 3.1, Sec. 3.3), the joint criterion (Eq. 9), the
 *     descending sort (Prop. 3.2), the calibration error (Eq. 3) and the acceptance rule (Eq. 10).
 *   - The producer of App. C (RMSNorm or adaptive LayerNorm with the channel reordering absorbed)
 *     with the NVFP4 quantizer attached: row statistics in fp32 over the original channel order,
 *     summed in the fixed 32-lane order stated at lane_order_sum.
 *   - PermuQuant-H (App. D): the Hadamard transform x H in fp32 with the stated butterfly order, its
 *     channels read through the permutation (x H P), then the NVFP4 quantizer.  The paper names the
 *     transform only; the matrix (Sylvester, times Paley's order-12 matrix for widths 12 * 2^n), the
 *     order of the additions and the 1/sqrt(K) scaling are readings stated at hadamard_row.
 *
 * Pins: see tests/test_oracle_*.py.  Every function here is pinned by hand-computed values,
 * closed forms, brute force on tiny inputs or an independent library routine, except the
 * behaviour of the whole pipeline on real-model activations ("parity unpinned": no weights,
 * calibration data or authors' code are available here; only synthetic stand-ins).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define PQO_CHUNK 16 /* rows per fp32 partial */
#define PQO_SLAB 128 /* rows per fp64 slab sum: 8 chunks, added in order starting from zero */

/* ------------------------------------------------------------------ scalar formats */

float pqo_bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> bf16, round to nearest even (finite inputs). */
uint16_t pqo_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t keep = u >> 16, rest = u & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;
    return (uint16_t)keep;
}

/* The eight E2M1 magnitudes, by 3-bit code (2 exponent bits, 1 mantissa bit). */
static const float E2M1_VALUE[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

float pqo_e2m1_value(uint8_t code) {
    float v = E2M1_VALUE[code & 7u];
    return (code & 8u) ? -v : v;
}

/* |y| -> 3-bit E2M1 code: nearest grid point, a tie goes to the neighbour whose mantissa bit
 * is 0 (codes 0, 2, 4, 6), anything above the top value saturates to 6. */
uint8_t pqo_e2m1_encode_abs(float ay) {
    for (int c = 0; c < 7; ++c) {
        float mid = 0.5f * (E2M1_VALUE[c] + E2M1_VALUE[c + 1]); /* exact */
        if (ay < mid) return (uint8_t)c;
        if (ay == mid) return (uint8_t)((c & 1) ? c + 1 : c);
    }
    return 7;
}

/* Unsigned E4M3 ("fn" flavour: bias 7, no infinity, 0x7F is the only NaN and never produced).
 * code = eeee mmm.  e = 0: subnormal 2^-6 * m/8.  e >= 1: 2^(e-7) * (1 + m/8).  Largest 448. */
float pqo_e4m3_value(uint8_t code) {
    int e = (code >> 3) & 15, m = code & 7;
    if (e == 0) return ldexpf((float)m, -9);
    return ldexpf((float)(8 + m), e - 10);
}

/* u >= 0 -> E4M3 code: nearest representable value, ties to the even code, saturating at 448. */
uint8_t pqo_e4m3_encode(float u) {
    for (int c = 0; c < 0x7E; ++c) {
        float lo = pqo_e4m3_value((uint8_t)c), hi = pqo_e4m3_value((uint8_t)(c + 1));
        float mid = 0.5f * (lo + hi); /* exact: both have 4 significant bits */
        if (u < mid) return (uint8_t)c;
        if (u == mid) return (uint8_t)((c & 1) ? c + 1 : c);
    }
    return 0x7E;
}

/* ------------------------------------------------------------------ tensor scale */

/* fp32 tensor scale from the tensor's absmax: absmax / (6 * 448); 1 for an all-zero tensor. */
float pqo_tensor_scale(const float *amax, int64_t K) {
    float a = 0.0f;
    for (int64_t i = 0; i < K; ++i)
        if (amax[i] > a) a = amax[i];
    if (a == 0.0f) return 1.0f;
    return a / 2688.0f;
}

/* ------------------------------------------------------------------ one group */

/* NVFP4: from the 16 (here: g) values of one group produce the scale byte, the decode scale d
 * and the 4-bit codes (sign bit = sign bit of the input, also for zeros). */
static void nvfp4_group(const float *x, int g, float ts, uint8_t *sf8_out, float *d_out,
                        uint8_t *code) {
    float amax = 0.0f;
    for (int j = 0; j < g; ++j) {
        float a = fabsf(x[j]);
        if (a > amax) amax = a;
    }
    float c = 6.0f * ts;
    float u = amax / c;
    uint8_t sf8 = pqo_e4m3_encode(u);
    float sf = pqo_e4m3_value(sf8);
    float d = sf * ts;
    float r = (d > 0.0f) ? 1.0f / d : 0.0f;
    for (int j = 0; j < g; ++j) {
        float y = x[j] * r;
        uint8_t mag = pqo_e2m1_encode_abs(fabsf(y));
        code[j] = (uint8_t)((signbit(x[j]) ? 8u : 0u) | mag);
    }
    *sf8_out = sf8;
    *d_out = d;
}

/* INT (Eq. 1-2): scale s = absmax / Q, z = clip(round(x / s)) with x / s evaluated as
 * x * fl(1/s), round = half-to-even. */
static void int_group(const float *x, int g, int Q, float *s_out, float *z) {
    float amax = 0.0f;
    for (int j = 0; j < g; ++j) {
        float a = fabsf(x[j]);
        if (a > amax) amax = a;
    }
    float s = amax / (float)Q;
    float r = (s > 0.0f) ? 1.0f / s : 0.0f;
    for (int j = 0; j < g; ++j) {
        float y = x[j] * r;
        float q = rintf(y); /* default rounding mode: nearest, ties to even */
        if (q > (float)Q) q = (float)Q;
        if (q < -(float)Q) q = -(float)Q;
        z[j] = q;
    }
    *s_out = s;
}

/* Squared error of one group, Eq. 3 restricted to the group: residual by one fused
 * multiply-add, squares summed in runs of eight ("octets"), octet sums combined by a balanced
 * adjacent-pair tree.  g <= 8: a single run.  Otherwise g/8 must be a power of two. */
static float group_sse(const float *x, const float *q, float d, int g) {
    float oct[64];
    int no = 0;
    for (int b = 0; b < g; b += 8) {
        float acc = 0.0f;
        int e = (b + 8 < g) ? b + 8 : g;
        for (int j = b; j < e; ++j) {
            float delta = fmaf(-q[j], d, x[j]);
            acc = fmaf(delta, delta, acc);
        }
        oct[no++] = acc;
    }
    while (no > 1) {
        for (int i = 0; i < no / 2; ++i) oct[i] = oct[2 * i] + oct[2 * i + 1];
        no /= 2;
    }
    return oct[0];
}

static int is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

static int format_ok(int kind, int bits, int group, int64_t K) {
    if (group <= 0 || K % group != 0) return 0;
    if (group > 8 && (group % 8 != 0 || !is_pow2(group / 8) || group > 512)) return 0;
    if (kind == 1 && (bits < 2 || bits > 8)) return 0;
    if (kind != 0 && kind != 1) return 0;
    return 1;
}

/* ------------------------------------------------------------------ column statistics */

/* Per channel i: sumsq[i] += sum_t x[t,i]^2 and amax[i] = max(amax[i], |x[t,i]|)  (second
 * moment of Assumption 3.1 before the division by the row count).  Rows are cut into slabs of
 * PQO_SLAB and slabs into chunks of PQO_CHUNK; inside a chunk the squares are added in fp32 in
 * row order, a slab's chunk partials are added in fp64 in ascending order starting from zero, and
 * the slab sums are added to the fp64 total in ascending order. */
int pqo_calib_stats(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, double *sumsq,
                    float *amax) {
    if (!T || !sumsq || !amax || rows <= 0 || K <= 0 || ld < K) return 1;
    for (int64_t s0 = 0; s0 < rows; s0 += PQO_SLAB) {
        int64_t s1 = (s0 + PQO_SLAB < rows) ? s0 + PQO_SLAB : rows;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < K; ++i) {
            double slab = 0.0;
            float a = amax[i];
            for (int64_t r0 = s0; r0 < s1; r0 += PQO_CHUNK) {
                int64_t r1 = (r0 + PQO_CHUNK < s1) ? r0 + PQO_CHUNK : s1;
                float p = 0.0f;
                for (int64_t t = r0; t < r1; ++t) {
                    float x = pqo_bf16_to_f32(T[t * ld + i]);
                    p = fmaf(x, x, p);
                    float ax = fabsf(x);
                    if (ax > a) a = ax;
                }
                slab += (double)p;
            }
            sumsq[i] += slab;
            amax[i] = a;
        }
    }
    return 0;
}

/* Per channel i: sum[i] += sum_t x[t,i]: the first moment the variance criterion of the reordering
 * ablation (Tab. 2(a)) needs beside the second one.  Same row blocking as pqo_calib_stats: fp32
 * additions in row order inside a chunk, a slab's chunk partials in fp64 from zero, slab sums into
 * the fp64 total, all in ascending order. */
int pqo_calib_sum(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, double *sum) {
    if (!T || !sum || rows <= 0 || K <= 0 || ld < K) return 1;
    for (int64_t s0 = 0; s0 < rows; s0 += PQO_SLAB) {
        int64_t s1 = (s0 + PQO_SLAB < rows) ? s0 + PQO_SLAB : rows;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < K; ++i) {
            double slab = 0.0;
            for (int64_t r0 = s0; r0 < s1; r0 += PQO_CHUNK) {
                int64_t r1 = (r0 + PQO_CHUNK < s1) ? r0 + PQO_CHUNK : s1;
                float p = 0.0f;
                for (int64_t t = r0; t < r1; ++t) p = p + pqo_bf16_to_f32(T[t * ld + i]);
                slab += (double)p;
            }
            sum[i] += slab;
        }
    }
    return 0;
}

/* Output-side calibration error, the other reading of "the quantization error on the
 * calibration data" of Sec. 3.3 (acceptance rule, Eq. 10): per output column n
 *     err[n] += sum_t (Yref[t,n] - Yq[t,n])^2
 * with Yref the unquantized product in fp32 and Yq the bf16 output of the quantized layer.  The
 * difference is one fp32 subtraction; the squares are summed over rows in chunks and slabs exactly
 * as in pqo_calib_stats. */
int pqo_output_error(const float *Yref, int64_t ld_ref, const uint16_t *Yq, int64_t ld_q, int64_t rows,
                     int64_t N, double *err) {
    if (!Yref || !Yq || !err || rows <= 0 || N <= 0 || ld_ref < N || ld_q < N) return 1;
    for (int64_t s0 = 0; s0 < rows; s0 += PQO_SLAB) {
        int64_t s1 = (s0 + PQO_SLAB < rows) ? s0 + PQO_SLAB : rows;
#pragma omp parallel for schedule(static)
        for (int64_t n = 0; n < N; ++n) {
            double slab = 0.0;
            for (int64_t r0 = s0; r0 < s1; r0 += PQO_CHUNK) {
                int64_t r1 = (r0 + PQO_CHUNK < s1) ? r0 + PQO_CHUNK : s1;
                float p = 0.0f;
                for (int64_t t = r0; t < r1; ++t) {
                    float d = Yref[t * ld_ref + n] - pqo_bf16_to_f32(Yq[t * ld_q + n]);
                    p = fmaf(d, d, p);
                }
                slab += (double)p;
            }
            err[n] += slab;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ permutation candidates */

typedef struct {
    double key;
    int32_t idx;
} keyed;

static int keyed_desc(const void *pa, const void *pb) {
    const keyed *a = (const keyed *)pa, *b = (const keyed *)pb;
    if (a->key > b->key) return -1;
    if (a->key < b->key) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx); /* equal keys: lower channel first */
}

/* Eq. 9 with alpha = j/J, j = 0..J:  v_i = (mu_a^2)^alpha (mu_w^2)^(1-alpha) is ordered like
 * v_i^J = (mu_a^2)^j (mu_w^2)^(J-j); that integer-power key is formed by left-to-right fp64
 * multiplication (j factors of a, then J-j factors of w, starting from 1).  Candidate j lists
 * the channels by descending key (Prop. 3.2), equal keys by ascending channel.
 * perms[j*K + pos] = channel read at position pos. */
int pqo_select_perm(const double *sumsq_a, int64_t rows_a, const double *sumsq_w, int64_t rows_w,
                    int64_t K, int J, int32_t *perms) {
    if (!sumsq_a || !sumsq_w || !perms || K <= 0 || J < 1 || rows_a <= 0 || rows_w <= 0) return 1;
    keyed *buf = (keyed *)malloc(sizeof(keyed) * (size_t)K);
    if (!buf) return 2;
    for (int j = 0; j <= J; ++j) {
        for (int64_t i = 0; i < K; ++i) {
            double a = sumsq_a[i] / (double)rows_a;
            double w = sumsq_w[i] / (double)rows_w;
            double key = 1.0;
            for (int f = 0; f < j; ++f) key = key * a;
            for (int f = 0; f < J - j; ++f) key = key * w;
            buf[i].key = key;
            buf[i].idx = (int32_t)i;
        }
        qsort(buf, (size_t)K, sizeof(keyed), keyed_desc); /* comparator is a total order */
        for (int64_t i = 0; i < K; ++i) perms[(int64_t)j * K + i] = buf[i].idx;
    }
    free(buf);
    return 0;
}

/* The absmax criterion of the reordering ablation (Tab. 2(a)): channels by descending absmax,
 * equal values by ascending channel.  perm[pos] = channel read at position pos. */
int pqo_order_by_absmax(const float *amax, int64_t K, int32_t *perm) {
    if (!amax || !perm || K <= 0) return 1;
    keyed *buf = (keyed *)malloc(sizeof(keyed) * (size_t)K);
    if (!buf) return 2;
    for (int64_t i = 0; i < K; ++i) {
        buf[i].key = (double)amax[i];
        buf[i].idx = (int32_t)i;
    }
    qsort(buf, (size_t)K, sizeof(keyed), keyed_desc);
    for (int64_t i = 0; i < K; ++i) perm[i] = buf[i].idx;
    free(buf);
    return 0;
}

/* The variance criterion of the reordering ablation (Tab. 2(a)): channels by descending
 * var_i = E[x_i^2] - E[x_i]^2 with E[x_i^2] = sumsq[i] / rows and E[x_i] = sum[i] / rows, all in fp64
 * (two divisions, one multiplication, one subtraction, no fused operation); equal values by
 * ascending channel.  The value may come out slightly negative for a constant channel; the order is
 * that of the signed values. */
int pqo_order_by_variance(const double *sum, const double *sumsq, int64_t rows, int64_t K, int32_t *perm) {
    if (!sum || !sumsq || !perm || K <= 0 || rows <= 0) return 1;
    keyed *buf = (keyed *)malloc(sizeof(keyed) * (size_t)K);
    if (!buf) return 2;
    for (int64_t i = 0; i < K; ++i) {
        double mean = sum[i] / (double)rows;
        double second = sumsq[i] / (double)rows;
        double sq = mean * mean;
        buf[i].key = second - sq;
        buf[i].idx = (int32_t)i;
    }
    qsort(buf, (size_t)K, sizeof(keyed), keyed_desc);
    for (int64_t i = 0; i < K; ++i) perm[i] = buf[i].idx;
    free(buf);
    return 0;
}

/* The "round-robin" order of the reordering ablation (Tab. 2(a)).  The paper names it without a
 * definition; the reading taken here: the channels, sorted by descending second moment (equal values by
 * ascending channel), are dealt to the K/g groups one at a time in turn, so that every group receives
 * channels of every magnitude (the opposite of clustering).  The channel of sorted rank r goes to group
 * r mod G at slot r div G, G = K / group:  perm[(r % G) * group + r / G] = sorted[r]. */
int pqo_order_round_robin(const double *sumsq, int64_t K, int group, int32_t *perm) {
    if (!sumsq || !perm || K <= 0 || group <= 0 || K % group != 0) return 1;
    keyed *buf = (keyed *)malloc(sizeof(keyed) * (size_t)K);
    if (!buf) return 2;
    for (int64_t i = 0; i < K; ++i) {
        buf[i].key = sumsq[i];
        buf[i].idx = (int32_t)i;
    }
    qsort(buf, (size_t)K, sizeof(keyed), keyed_desc);
    int64_t G = K / group;
    for (int64_t r = 0; r < K; ++r) perm[(r % G) * group + r / G] = buf[r].idx;
    free(buf);
    return 0;
}

/* ------------------------------------------------------------------ calibration error */

/* Eq. 3 on one batch: for every candidate order p and group column k,
 *   err[p*Kg + k] += sum_t || e - e_hat ||^2  with  e_j = T[t, perm_p(k*g + j)].
 * kind 0 = NVFP4 (bits ignored, ts used), kind 1 = INT (bits, ts ignored).
 * perms == NULL means one candidate, the identity.  Rows in slabs and chunks as in
 * pqo_calib_stats. */
int pqo_group_error(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, int kind, int bits,
                    int group, float ts, const int32_t *perms, int P, double *err) {
    if (!T || !err || rows <= 0 || K <= 0 || ld < K || P < 1) return 1;
    if (!format_ok(kind, bits, group, K)) return 1;
    const int g = group;
    const int64_t Kg = K / g;
    const int Q = (1 << (bits - 1)) - 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int p = 0; p < P; ++p) {
        for (int64_t k = 0; k < Kg; ++k) {
            const int32_t *perm = perms ? perms + (int64_t)p * K : NULL;
            float x[512], q[512];
            uint8_t code[512];
            double total = err[(int64_t)p * Kg + k], slab = 0.0;
            for (int64_t r0 = 0; r0 < rows; r0 += PQO_CHUNK) {
                int64_t r1 = (r0 + PQO_CHUNK < rows) ? r0 + PQO_CHUNK : rows; /* PQO_SLAB % PQO_CHUNK == 0 */
                if (r0 % PQO_SLAB == 0) slab = 0.0;
                float part = 0.0f;
                for (int64_t t = r0; t < r1; ++t) {
                    for (int j = 0; j < g; ++j) {
                        int64_t ch = perm ? perm[k * g + j] : k * g + j;
                        x[j] = pqo_bf16_to_f32(T[t * ld + ch]);
                    }
                    float d;
                    if (kind == 0) {
                        uint8_t sf8;
                        nvfp4_group(x, g, ts, &sf8, &d, code);
                        for (int j = 0; j < g; ++j) q[j] = pqo_e2m1_value(code[j]);
                    } else {
                        int_group(x, g, Q, &d, q);
                    }
                    part = part + group_sse(x, q, d, g);
                }
                slab += (double)part;
                if (r1 % PQO_SLAB == 0 || r1 == rows) total += slab;
            }
            err[(int64_t)p * Kg + k] = total;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ selection + acceptance */

/* E_p = lambda_x * sum_k err_x[p,k] + lambda_w * sum_k err_w[p,k]   (p = 0: original order).
 * best = candidate in 1..P with the smallest E (first on ties).
 * Eq. 10 in multiplicative form: accept iff E_0 - E_best > tau * E_0  (strict). */
int pqo_accept(const double *err_x, double lambda_x, const double *err_w, double lambda_w, int P,
               int64_t Kg, double tau, int32_t *best, int32_t *accept, double *E) {
    if (!err_x || !err_w || !best || !accept || P < 1 || Kg <= 0) return 1;
    double E0 = 0.0, Ebest = 0.0;
    int32_t b = 1;
    for (int p = 0; p <= P; ++p) {
        double sx = 0.0, sw = 0.0;
        for (int64_t k = 0; k < Kg; ++k) sx = sx + err_x[(int64_t)p * Kg + k];
        for (int64_t k = 0; k < Kg; ++k) sw = sw + err_w[(int64_t)p * Kg + k];
        double tx = lambda_x * sx;
        double tw = lambda_w * sw;
        double Ep = tx + tw;
        if (E) E[p] = Ep;
        if (p == 0) E0 = Ep;
        else if (p == 1 || Ep < Ebest) {
            Ebest = Ep;
            b = p;
        }
    }
    double gain = E0 - Ebest;
    double need = tau * E0;
    *best = b;
    *accept = (gain > need) ? 1 : 0;
    return 0;
}

/* Default weights: each side's error relative to its own energy, 1 / sum_i sumsq[i]. */
double pqo_error_weight(const double *sumsq, int64_t K) {
    double s = 0.0;
    for (int64_t i = 0; i < K; ++i) s = s + sumsq[i];
    return 1.0 / s;
}

/* ------------------------------------------------------------------ NVFP4 quantize */

/* codes[r, j/2] (even channel in the low nibble) and sf[r, j/16] for the tensor read through the
 * gather out[:, j] = T[:, perm[j]]  (perm == NULL: identity).  Scale bytes in plain row-major
 * order [rows, K/16]. */
int pqo_quant_nvfp4(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, const int32_t *perm,
                    float ts, uint8_t *codes, uint8_t *sf) {
    if (!T || !codes || !sf || rows <= 0 || K <= 0 || K % 16 != 0 || ld < K) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < rows; ++t) {
        for (int64_t k = 0; k < K / 16; ++k) {
            float x[16], d;
            uint8_t code[16], sf8;
            for (int j = 0; j < 16; ++j) {
                int64_t ch = perm ? perm[k * 16 + j] : k * 16 + j;
                x[j] = pqo_bf16_to_f32(T[t * ld + ch]);
            }
            nvfp4_group(x, 16, ts, &sf8, &d, code);
            sf[t * (K / 16) + k] = sf8;
            for (int j = 0; j < 16; j += 2)
                codes[t * (K / 2) + (k * 16 + j) / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ fused norm + reorder + quantize */

/* Sum over a row in the order a 32-lane row walk gives: element i belongs to lane (i / 8) % 32,
 * each lane adds its elements in ascending i, the 32 lane partials are then combined by a
 * butterfly (strides 16, 8, 4, 2, 1; every lane ends with the same value).
 * mode 0: sum of v[i];  mode 1: sum of v[i]^2 by fused multiply-add. */
static float lane_order_sum(const float *v, int64_t K, int mode) {
    float p[32], q[32];
    for (int l = 0; l < 32; ++l) p[l] = 0.0f;
    for (int64_t i = 0; i < K; ++i) {
        int l = (int)((i / 8) % 32);
        p[l] = mode ? fmaf(v[i], v[i], p[l]) : p[l] + v[i];
    }
    for (int m = 16; m >= 1; m >>= 1) {
        for (int l = 0; l < 32; ++l) q[l] = p[l] + p[l ^ m];
        for (int l = 0; l < 32; ++l) p[l] = q[l];
    }
    return p[0];
}

/* Normalization with the channel reordering and the NVFP4 quantizer behind it (the absorbed
 * permutation of App. C, with the quantizer of Eq. 8 attached): per row x of H and output position j
 * reading channel c = perm[j]
 *   kind 0 (RMSNorm):            out_j = (x_c * inv) * a_j,                   inv = 1 / sqrt(mean(x^2) + eps)
 *   kind 1 (adaptive LayerNorm): out_j = fma((x_c - mu) * inv, 1 + a_j, b_j), inv = 1 / sqrt(mean((x - mu)^2) + eps)
 * a (weight or modulation scale) and b (modulation shift) are indexed by OUTPUT position: they
 * arrive reordered, (1 + Ps) and Pb of App. C.  The statistics run over the ORIGINAL channel order,
 * so they do not depend on the permutation.  Then the NVFP4 groups of out.  y_bf16 (optional)
 * receives bf16(out), the tensor the unfused kernel of App. C would write.
 * All arithmetic fp32, sums in lane order (lane_order_sum). */
int pqo_norm_quant_nvfp4(const uint16_t *H, int64_t rows, int64_t K, int64_t ld, int kind, const float *a,
                         const float *b, float eps, const int32_t *perm, float ts, uint8_t *codes,
                         uint8_t *sf, uint16_t *y_bf16) {
    if (!H || !a || !codes || !sf || rows <= 0 || K <= 0 || K % 16 != 0 || ld < K) return 1;
    if (kind != 0 && kind != 1) return 1;
    if (kind == 1 && !b) return 1;
    int fail = 0;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < rows; ++t) {
        float *x = (float *)malloc(sizeof(float) * (size_t)K * 2);
        if (!x) {
            fail = 1;
            continue;
        }
        float *y = x + K;
        float mu = 0.0f, inv;
        for (int64_t i = 0; i < K; ++i) x[i] = pqo_bf16_to_f32(H[t * ld + i]);
        if (kind == 0) {
            float ms = lane_order_sum(x, K, 1) / (float)K;
            inv = 1.0f / sqrtf(ms + eps);
        } else {
            mu = lane_order_sum(x, K, 0) / (float)K;
            for (int64_t i = 0; i < K; ++i) y[i] = x[i] - mu;
            float var = lane_order_sum(y, K, 1) / (float)K;
            inv = 1.0f / sqrtf(var + eps);
        }
        for (int64_t k = 0; k < K / 16; ++k) {
            float g[16], d;
            uint8_t code[16], sf8;
            for (int j = 0; j < 16; ++j) {
                int64_t pos = k * 16 + j, c = perm ? perm[pos] : pos;
                g[j] = (kind == 0) ? (x[c] * inv) * a[pos] : fmaf((x[c] - mu) * inv, 1.0f + a[pos], b[pos]);
            }
            nvfp4_group(g, 16, ts, &sf8, &d, code);
            sf[t * (K / 16) + k] = sf8;
            for (int j = 0; j < 16; j += 2)
                codes[t * (K / 2) + (k * 16 + j) / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
            if (y_bf16)
                for (int j = 0; j < 16; ++j) y_bf16[t * K + k * 16 + j] = pqo_f32_to_bf16(g[j]);
        }
        free(x);
    }
    return fail;
}

/* ------------------------------------------------------------------ PermuQuant-H: Hadamard, reorder, quantize */

/* Legendre symbol modulo 11: 0 for 0, +1 for the non-zero squares {1, 3, 4, 5, 9}, -1 otherwise. */
static int legendre11(int r) {
    r = ((r % 11) + 11) % 11;
    if (r == 0) return 0;
    for (int t = 1; t < 11; ++t)
        if ((t * t) % 11 == r) return 1;
    return -1;
}

/* The Hadamard matrix of order 12 by Paley's first construction for q = 11 (q = 3 mod 4):
 * H = I + S with the skew matrix S = [[0, 1...1], [-1...-1 (column), Q]], Q[i][j] = chi(i - j). */
static int hadamard12_entry(int i, int j) {
    if (i == j) return 1;
    if (i == 0) return 1;
    if (j == 0) return -1;
    return legendre11((i - 1) - (j - 1));
}

/* Which widths the transform is defined for here: K = 2^n (m = 1), or K = 12 * 2^n (m = 12). */
static int hadamard_factor(int64_t K) {
    if (K <= 0) return 0;
    if ((K & (K - 1)) == 0) return 1;
    if (K % 12 == 0 && ((K / 12) & (K / 12 - 1)) == 0) return 12;
    return 0;
}

/* One row x[K] (in place): y = x (H_m (x) H_{2^n}) / sqrt(K), i.e. with the channel index written
 * i = a * 2^n + b the matrix entry is H_m[a][a'] * (-1)^popcount(b & b').  fp32 throughout, in this
 * order: (1) for m = 12, across the 12 segments: u[a'][b] = sum_a x[a][b] * H12[a][a'], the terms
 * added one by one in ascending a (the first term is +-x[0][b] itself); (2) inside every segment the
 * in-place butterflies of the fast Walsh-Hadamard transform, strides 1, 2, 4, ..., 2^(n-1):
 * (x[i], x[i+h]) <- (x[i] + x[i+h], x[i] - x[i+h]) for every i with bit h clear; (3) one
 * multiplication by fl(1 / sqrt(K)) (the double-precision value rounded to fp32). */
static void hadamard_row(float *x, int64_t K, float *tmp) {
    int m = hadamard_factor(K);
    int64_t seg = K / m;
    if (m == 12) {
        for (int64_t b = 0; b < seg; ++b)
            for (int ap = 0; ap < 12; ++ap) {
                float acc = (hadamard12_entry(0, ap) > 0) ? x[b] : -x[b];
                for (int a = 1; a < 12; ++a) {
                    float v = x[a * seg + b];
                    acc = (hadamard12_entry(a, ap) > 0) ? acc + v : acc - v;
                }
                tmp[ap * seg + b] = acc;
            }
        memcpy(x, tmp, sizeof(float) * (size_t)K);
    }
    for (int a = 0; a < m; ++a) {
        float *s = x + a * seg;
        for (int64_t h = 1; h < seg; h <<= 1)
            for (int64_t i = 0; i < seg; ++i)
                if (!(i & h)) {
                    float p = s[i], q = s[i + h];
                    s[i] = p + q;
                    s[i + h] = p - q;
                }
    }
    float scale = (float)(1.0 / sqrt((double)K));
    for (int64_t i = 0; i < K; ++i) x[i] = x[i] * scale;
}

/* PermuQuant-H runtime producer (App. D): the Hadamard transform of every row, its channels read in
 * the order `perm` (x H P: position j takes transformed channel perm[j]; NULL = transformed order),
 * then the NVFP4 groups of that, quantized from the fp32 values.  codes / sf may be NULL (transform
 * only); y_bf16 (optional) receives bf16 of the reordered transformed row, y_f32 (optional) the fp32
 * values themselves.  Returns 2 for a width the transform is not defined for. */
int pqo_hadamard_quant_nvfp4(const uint16_t *X, int64_t rows, int64_t K, int64_t ld, const int32_t *perm, float ts,
                             uint8_t *codes, uint8_t *sf, uint16_t *y_bf16, float *y_f32) {
    if (!X || rows <= 0 || K <= 0 || K % 16 != 0 || ld < K) return 1;
    if ((codes == NULL) != (sf == NULL)) return 1;
    if (!hadamard_factor(K)) return 2;
    int fail = 0;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < rows; ++t) {
        float *x = (float *)malloc(sizeof(float) * (size_t)K * 2);
        if (!x) {
            fail = 1;
            continue;
        }
        for (int64_t i = 0; i < K; ++i) x[i] = pqo_bf16_to_f32(X[t * ld + i]);
        hadamard_row(x, K, x + K);
        for (int64_t k = 0; k < K / 16; ++k) {
            float g[16], d;
            uint8_t code[16], sf8;
            for (int j = 0; j < 16; ++j) {
                int64_t pos = k * 16 + j;
                g[j] = x[perm ? perm[pos] : pos];
                if (y_bf16) y_bf16[t * K + pos] = pqo_f32_to_bf16(g[j]);
                if (y_f32) y_f32[t * K + pos] = g[j];
            }
            if (codes) {
                nvfp4_group(g, 16, ts, &sf8, &d, code);
                sf[t * (K / 16) + k] = sf8;
                for (int j = 0; j < 16; j += 2)
                    codes[t * (K / 2) + (k * 16 + j) / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
            }
        }
        free(x);
    }
    return fail;
}

/* Decode one NVFP4 tensor back to fp32: value * (scale * ts), both products in fp32. */
int pqo_dequant_nvfp4(const uint8_t *codes, const uint8_t *sf, float ts, int64_t rows, int64_t K,
                      float *out) {
    if (!codes || !sf || !out || K % 16 != 0) return 1;
    for (int64_t t = 0; t < rows; ++t)
        for (int64_t j = 0; j < K; ++j) {
            uint8_t b = codes[t * (K / 2) + j / 2];
            uint8_t c = (j & 1) ? (uint8_t)(b >> 4) : (uint8_t)(b & 15u);
            float d = pqo_e4m3_value(sf[t * (K / 16) + j / 16]) * ts;
            out[t * K + j] = pqo_e2m1_value(c) * d;
        }
    return 0;
}

/* ------------------------------------------------------------------ INT fake-quant */

/* Eq. 1-2 followed by rounding the dequantized value to bf16; optional gather as above. */
int pqo_fakequant_int(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, int bits, int group,
                      const int32_t *perm, uint16_t *out, int64_t ldo) {
    if (!T || !out || rows <= 0 || ld < K || ldo < K) return 1;
    if (!format_ok(1, bits, group, K)) return 1;
    const int g = group, Q = (1 << (bits - 1)) - 1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < rows; ++t) {
        float x[512], z[512];
        for (int64_t k = 0; k < K / g; ++k) {
            float s;
            for (int j = 0; j < g; ++j) {
                int64_t ch = perm ? perm[k * g + j] : k * g + j;
                x[j] = pqo_bf16_to_f32(T[t * ld + ch]);
            }
            int_group(x, g, Q, &s, z);
            for (int j = 0; j < g; ++j) out[t * ldo + k * g + j] = pqo_f32_to_bf16(z[j] * s);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ GEMM reference */

static double dq_elem(const uint8_t *codes, const uint8_t *sf, int64_t K, int64_t row, int64_t j) {
    uint8_t b = codes[row * (K / 2) + j / 2];
    uint8_t c = (j & 1) ? (uint8_t)(b >> 4) : (uint8_t)(b & 15u);
    return (double)pqo_e2m1_value(c) * (double)pqo_e4m3_value(sf[row * (K / 16) + j / 16]);
}

/* Eq. 8's right-hand side on dequantized operands, in fp64:
 *   Y[m,n] = ts_x * ts_w * sum_k dq_x[m,k] * dq_w[n,k],  dq = E2M1 value * E4M3 scale. */
double pqo_gemm_ref_one(const uint8_t *xq, const uint8_t *sfx, float ts_x, const uint8_t *wq,
                        const uint8_t *sfw, float ts_w, int64_t K, int64_t m, int64_t n) {
    double acc = 0.0;
    for (int64_t k = 0; k < K; ++k) acc += dq_elem(xq, sfx, K, m, k) * dq_elem(wq, sfw, K, n, k);
    return (double)ts_x * (double)ts_w * acc;
}

/* All of Y (row-major [M,N], fp64). */
int pqo_gemm_ref(const uint8_t *xq, const uint8_t *sfx, float ts_x, const uint8_t *wq,
                 const uint8_t *sfw, float ts_w, int64_t M, int64_t N, int64_t K, double *Y) {
    if (!xq || !sfx || !wq || !sfw || !Y || K % 16 != 0) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n)
            Y[m * N + n] = pqo_gemm_ref_one(xq, sfx, ts_x, wq, sfw, ts_w, K, m, n);
    return 0;
}

/* Selected entries only: out[i] = Y[ms[i], ns[i]]. */
int pqo_gemm_ref_sampled(const uint8_t *xq, const uint8_t *sfx, float ts_x, const uint8_t *wq,
                         const uint8_t *sfw, float ts_w, int64_t K, const int64_t *ms,
                         const int64_t *ns, int64_t count, double *out) {
    if (!xq || !sfx || !wq || !sfw || !ms || !ns || !out || K % 16 != 0) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i)
        out[i] = pqo_gemm_ref_one(xq, sfx, ts_x, wq, sfw, ts_w, K, ms[i], ns[i]);
    return 0;
}

/* The unquantized product of Eq. 8's left-hand side, fp64, for function-preservation checks:
 * Y[m,n] = sum_k X[m, perm[k]] * Wt[n, perm[k]]. */
int pqo_gemm_bf16_ref(const uint16_t *X, const uint16_t *Wt, int64_t M, int64_t N, int64_t K,
                      const int32_t *perm, double *Y) {
    if (!X || !Wt || !Y) return 1;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                int64_t ch = perm ? perm[k] : k;
                acc += (double)pqo_bf16_to_f32(X[m * K + ch]) * (double)pqo_bf16_to_f32(Wt[n * K + ch]);
            }
            Y[m * N + n] = acc;
        }
    return 0;
}

int pqo_chunk_rows(void) { return PQO_CHUNK; }
int pqo_slab_rows(void) { return PQO_SLAB; }

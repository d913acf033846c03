/*
 * S-STE oracle: a plain, slow, CPU-only statement of what the sparse linear
 * layer's hot path computes.  TEST INFRASTRUCTURE ONLY: nothing on the product
 * path may link, load or call this file.  It shares no code with the CUDA
 * library; every function below is written from the paper's definitions.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC sste_oracle.c -lm
 * (-ffp-contract=off: every fp32 step below is one IEEE-754 operation, so a
 * GPU that performs the same steps without FMA contraction gets the same bits.)
 *
 * Parity pins live in tests/test_oracle_*.py.  The GEMMs of the path are not
 * here: they are numpy fp64 matmuls in oracle/sste_oracle.py.
 *
 * Formats
 *   bf16 tensors are uint16_t bit patterns, fp8 tensors uint8_t bit patterns.
 *   odt: 0 = bf16 output values, 2 = E4M3 (forward operands), 3 = E5M2 (gradients).
 *   Canonical compressed format of a [rows, K] 2:4 matrix (K % 16 == 0):
 *     vals[r, 2g + {0,1}]  the two kept values of group g (elements 4g..4g+3 of row r)
 *                          in ascending position order,
 *     meta[r, g/4]         uint16_t; the nibble of group g sits at bits [4(g%4), 4(g%4)+4)
 *                          and is p0 | (p1 << 2) with p0 < p1 the kept positions.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------ codecs */

static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even fp32 -> bf16; NaN stays NaN (quiet) */
static uint16_t f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/*
 * Generic "round to nearest even, saturate to the largest finite value" encoder
 * for a small binary float with ebits exponent bits, mbits mantissa bits and the
 * given bias; maxv is the largest finite value of the format (448 for E4M3 in its
 * "fn" flavour, 57344 for E5M2).  NaN maps to the format's canonical NaN.
 * FP8 whole-process training: Section 5.2.
 */
static uint8_t fp8_encode(float x, int ebits, int mbits, int bias, double maxv, uint8_t nan_code)
{
    uint8_t sign = signbit(x) ? 0x80u : 0u;
    if (isnan(x)) return (uint8_t)(sign | nan_code);
    double a = fabs((double)x);
    if (a == 0.0) return sign;
    if (a > maxv) a = maxv;                 /* satfinite (also catches +-inf) */
    int e;
    (void)frexp(a, &e);                     /* a = f * 2^e, f in [0.5, 1) */
    e -= 1;                                 /* a in [2^e, 2^(e+1)) */
    int emin = 1 - bias;                    /* exponent of the smallest normal */
    if (e < emin) e = emin;                 /* subnormal range shares the quantum of emin */
    double quantum = ldexp(1.0, e - mbits);
    double q = nearbyint(a / quantum);      /* default rounding mode: ties to even */
    double v = q * quantum;
    if (v > maxv) v = maxv;
    if (v == 0.0) return sign;
    /* encode v exactly */
    int e2;
    (void)frexp(v, &e2);
    e2 -= 1;
    uint32_t efield, mfield;
    if (e2 < emin) {
        efield = 0;
        mfield = (uint32_t)(v / ldexp(1.0, emin - mbits));
    } else {
        efield = (uint32_t)(e2 + bias);
        mfield = (uint32_t)(v / ldexp(1.0, e2 - mbits)) - (1u << mbits);
    }
    (void)ebits;
    return (uint8_t)(sign | (efield << mbits) | mfield);
}

static uint8_t f32_to_e4m3(float x) { return fp8_encode(x, 4, 3, 7, 448.0, 0x7f); }
static uint8_t f32_to_e5m2(float x) { return fp8_encode(x, 5, 2, 15, 57344.0, 0x7f); }

static float e4m3_to_f32(uint8_t c)
{
    int s = c >> 7, e = (c >> 3) & 0xf, m = c & 7;
    double v;
    if (e == 0xf && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);            /* m/8 * 2^-6 */
    else v = ldexp(1.0 + m / 8.0, e - 7);
    return (float)(s ? -v : v);
}

static float e5m2_to_f32(uint8_t c)
{
    int s = c >> 7, e = (c >> 2) & 0x1f, m = c & 3;
    double v;
    if (e == 0x1f) return m ? NAN : (s ? -INFINITY : INFINITY);
    if (e == 0) v = ldexp((double)m, -16);           /* m/4 * 2^-14 */
    else v = ldexp(1.0 + m / 4.0, e - 15);
    return (float)(s ? -v : v);
}

void sste_oracle_bf16_to_f32(const uint16_t *in, int64_t n, float *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_f32(in[i]);
}
void sste_oracle_f32_to_bf16(const float *in, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16(in[i]);
}
void sste_oracle_f32_to_fp8(const float *in, int64_t n, int odt, uint8_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = (odt == 2) ? f32_to_e4m3(in[i]) : f32_to_e5m2(in[i]);
}
void sste_oracle_fp8_to_f32(const uint8_t *in, int64_t n, int dt, float *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = (dt == 2) ? e4m3_to_f32(in[i]) : e5m2_to_f32(in[i]);
}

static void store_val(void *base, int64_t idx, float v, int odt)
{
    if (odt == 0) ((uint16_t *)base)[idx] = f32_to_bf16(v);
    else if (odt == 2) ((uint8_t *)base)[idx] = f32_to_e4m3(v);
    else ((uint8_t *)base)[idx] = f32_to_e5m2(v);
}

/* ------------------------------------------------ S_soft, Eq. (4) (Sec. 4.1) */

/*
 * One group of four: t is the second-smallest magnitude (t = |t2| with
 * |t1|<=|t2|<=|t3|<=|t4|); each element moves towards zero by t and elements
 * with |a_i| <= t become +0.  s_i = sign(a_i) * (|a_i| - t) evaluated as ONE
 * fp32 subtraction of the magnitudes.
 */
static void s_soft_group(const float a[4], float s[4])
{
    float m[4], sorted[4];
    for (int i = 0; i < 4; ++i) m[i] = fabsf(a[i]);
    memcpy(sorted, m, sizeof sorted);
    for (int i = 1; i < 4; ++i)                 /* insertion sort, ascending */
        for (int j = i; j > 0 && sorted[j - 1] > sorted[j]; --j) {
            float tmp = sorted[j]; sorted[j] = sorted[j - 1]; sorted[j - 1] = tmp;
        }
    float t = sorted[1];
    for (int i = 0; i < 4; ++i) {
        float d = m[i] - t;
        s[i] = (d > 0.0f) ? copysignf(d, a[i]) : 0.0f;
    }
}

/* S_soft of a bf16 [O, I] matrix, groups of 4 along I; result as fp32 */
void sste_oracle_s_soft(const uint16_t *W, int O, int I, float *S)
{
    for (int64_t r = 0; r < O; ++r)
        for (int g = 0; g < I / 4; ++g) {
            float a[4], s[4];
            for (int i = 0; i < 4; ++i) a[i] = bf16_to_f32(W[r * I + 4 * g + i]);
            s_soft_group(a, s);
            for (int i = 0; i < 4; ++i) S[r * I + 4 * g + i] = s[i];
        }
}

/* ---------------------------------------- beta, Eq. (5) (Sec. 4.2, "Minimizing MSE") */

/*
 * beta = <w, S_soft(w)> / ||S_soft(w)||^2 with S_soft evaluated in exact real
 * arithmetic (fp64 on bf16 inputs) and fp64 sums.  num/den are returned too.
 * A zero denominator (S_soft(w) == 0) returns beta = 1 and *degenerate = 1.
 */
double sste_oracle_beta(const uint16_t *W, int O, int I, double *num_out, double *den_out, int *degenerate)
{
    double num = 0.0, den = 0.0;
    for (int64_t r = 0; r < O; ++r)
        for (int g = 0; g < I / 4; ++g) {
            double a[4], m[4], sorted[4];
            for (int i = 0; i < 4; ++i) {
                a[i] = (double)bf16_to_f32(W[r * I + 4 * g + i]);
                m[i] = fabs(a[i]);
                sorted[i] = m[i];
            }
            for (int i = 1; i < 4; ++i)
                for (int j = i; j > 0 && sorted[j - 1] > sorted[j]; --j) {
                    double tmp = sorted[j]; sorted[j] = sorted[j - 1]; sorted[j - 1] = tmp;
                }
            double t = sorted[1];
            for (int i = 0; i < 4; ++i) {
                double d = m[i] - t;
                if (d > 0.0) {
                    double s = copysign(d, a[i]);
                    num += a[i] * s;
                    den += s * s;
                }
            }
        }
    if (num_out) *num_out = num;
    if (den_out) *den_out = den;
    if (degenerate) *degenerate = (den == 0.0);
    return (den == 0.0) ? 1.0 : num / den;
}

/* ------------------------------------- kept positions of a group (compression) */

/*
 * The two kept positions of a group given the four magnitudes: rank by
 * (magnitude descending, index ascending) and keep the first two.  Every
 * element with a nonzero S_soft output is among them (at most two magnitudes
 * exceed the second-smallest).  Returns p0 < p1.
 */
static void kept_pair(const float m[4], int *p0, int *p1)
{
    int keep[4] = {0, 0, 0, 0};
    for (int i = 0; i < 4; ++i) {
        int rank = 0;
        for (int j = 0; j < 4; ++j)
            if (m[j] > m[i] || (m[j] == m[i] && j < i)) ++rank;
        keep[i] = rank < 2;
    }
    int first = -1, second = -1;
    for (int i = 0; i < 4; ++i)
        if (keep[i]) { if (first < 0) first = i; else second = i; }
    *p0 = first; *p1 = second;
}

/*
 * Steps (1) of the training iteration (Sec. 2) with S = beta * S_soft (Sec. 4):
 * w~ = fl32(s * beta) [ * wscale for FP8 ], one RNE cast to odt, compressed to the
 * canonical format.  dense (nullable) receives the uncompressed w~ [O, I] in odt.
 */
void sste_oracle_project_compress(const uint16_t *W, int O, int I, float beta, float wscale, int odt,
                                  void *vals, uint16_t *meta, void *dense)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < O; ++r) {
        for (int g = 0; g < I / 4; ++g) {
            float a[4], m[4], s[4], w[4];
            for (int i = 0; i < 4; ++i) { a[i] = bf16_to_f32(W[r * I + 4 * g + i]); m[i] = fabsf(a[i]); }
            s_soft_group(a, s);
            for (int i = 0; i < 4; ++i) {
                w[i] = s[i] * beta;
                if (odt != 0) w[i] = w[i] * wscale;
                if (s[i] == 0.0f) w[i] = 0.0f;            /* pruned entries are canonical +0 */
            }
            int p0, p1;
            kept_pair(m, &p0, &p1);
            store_val(vals, r * (I / 2) + 2 * g + 0, w[p0], odt);
            store_val(vals, r * (I / 2) + 2 * g + 1, w[p1], odt);
            uint16_t nib = (uint16_t)(p0 | (p1 << 2));
            int64_t mi = r * (I / 16) + g / 4;
            if (g % 4 == 0) meta[mi] = 0;
            meta[mi] |= (uint16_t)(nib << (4 * (g % 4)));
            if (dense)
                for (int i = 0; i < 4; ++i) store_val(dense, r * I + 4 * g + i, w[i], odt);
        }
    }
}

/* canonical compressed [rows, K/2] + meta -> dense fp32 [rows, K] */
void sste_oracle_decompress(const void *vals, const uint16_t *meta, int rows, int K, int dt, float *dense)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int g = 0; g < K / 4; ++g) {
            int nib = (meta[r * (K / 16) + g / 4] >> (4 * (g % 4))) & 0xf;
            int p0 = nib & 3, p1 = (nib >> 2) & 3;
            float v[2];
            for (int j = 0; j < 2; ++j) {
                int64_t idx = r * (K / 2) + 2 * g + j;
                if (dt == 0) v[j] = bf16_to_f32(((const uint16_t *)vals)[idx]);
                else if (dt == 2) v[j] = e4m3_to_f32(((const uint8_t *)vals)[idx]);
                else v[j] = e5m2_to_f32(((const uint8_t *)vals)[idx]);
            }
            for (int i = 0; i < 4; ++i) dense[r * K + 4 * g + i] = 0.0f;
            dense[r * K + 4 * g + p0] = v[0];
            dense[r * K + 4 * g + p1] = v[1];
        }
}

/* --------------------------------------------------------- Philox4x32-10 */

void sste_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ------------------------------------------- MVUE 2:4 of dY (Sec. 5.1) */

/*
 * Minimum-variance unbiased 2:4 estimator of one group a[0..3] given a uniform
 * u in [0,1) (a multiple of 2^-24).  Inclusion probabilities p_i = min(1, c|a_i|)
 * with sum 2; a kept element carries a_i / p_i.  With x the first largest
 * magnitude and rest the sum of the other three:
 *   clipped   (m_x >= rest): keep x as is, and one other j with prob m_j/rest, value sign(a_j)*rest;
 *   unclipped (m_x <  rest): p_i = 2 m_i / S; systematic sampling with the two
 *                            points u*S/2 and u*S/2 + S/2 on the cumulative sums; both values sign*S/2.
 * All arithmetic is fp32, one rounding per operation, in the order written.
 * Outputs: kept positions q0 < q1 and their fp32 values (before the cast).
 */
static void mvue_group(const float a[4], float u, int *q0, int *q1, float *v0, float *v1)
{
    float m[4];
    for (int i = 0; i < 4; ++i) m[i] = fabsf(a[i]);
    int x = 0;
    for (int i = 1; i < 4; ++i) if (m[i] > m[x]) x = i;   /* first argmax */
    int o[3], n = 0;
    for (int i = 0; i < 4; ++i) if (i != x) o[n++] = i;
    float rest = (m[o[0]] + m[o[1]]) + m[o[2]];
    int ja, jb;
    float va, vb;
    if (m[x] >= rest) {
        int second;
        float val;
        if (rest == 0.0f) {
            second = o[0];
            val = 0.0f;
        } else {
            float r = u * rest;
            float c0 = m[o[0]];
            float c1 = c0 + m[o[1]];
            second = (c0 > r) ? o[0] : (c1 > r) ? o[1] : o[2];
            if (m[second] == 0.0f) {            /* only reachable through rounding of c1 / r */
                for (int k = 2; k >= 0; --k) if (m[o[k]] > 0.0f) { second = o[k]; break; }
            }
            val = copysignf(rest, a[second]);
        }
        ja = x; va = a[x];
        jb = second; vb = val;
    } else {
        float c0 = m[0];
        float c1 = c0 + m[1];
        float c2 = c1 + m[2];
        float c3 = c2 + m[3];
        float c[4] = {c0, c1, c2, c3};
        float half = 0.5f * c3;
        float r1 = u * half;
        float r2 = r1 + half;
        int j1 = 3;
        for (int i = 0; i < 4; ++i) if (c[i] > r1) { j1 = i; break; }
        int j2 = 3;
        for (int i = j1 + 1; i < 4; ++i) if (c[i] > r2) { j2 = i; break; }
        if (j1 == 3) { j1 = 2; j2 = 3; }        /* only reachable through rounding */
        ja = j1; va = copysignf(half, a[j1]);
        jb = j2; vb = copysignf(half, a[j2]);
    }
    if (ja < jb) { *q0 = ja; *v0 = va; *q1 = jb; *v1 = vb; }
    else         { *q0 = jb; *v0 = vb; *q1 = ja; *v1 = va; }
}

/* exported single-group form (for the statistical pins) */
void sste_oracle_mvue_group(const float a[4], float u, int pos[2], float val[2])
{
    mvue_group(a, u, &pos[0], &pos[1], &val[0], &val[1]);
}

/*
 * MVUE(dY^T): dY is [T, O] bf16 row-major; groups are 4 consecutive tokens of
 * one column j.  Group (j, tg) has global index g = (tg_offset + tg)*O + j (tg_offset = token groups
 * that precede this dY in the whole batch; 0 unless the batch is sharded); Philox counter
 * (q_lo, q_hi, tensor_id, step) with q = g>>2, key (seed_lo, seed_hi); the group
 * uses output word g&3, top 24 bits, u = k * 2^-24.
 * Output is the canonical compressed format of the TRANSPOSED matrix: rows = O,
 * K = T: gvals[j, 2*tg + {0,1}], gmeta[j, tg/4].  FP8: values are cast as
 * E5M2(fl32(v * gscale)); dense_q (nullable) receives E5M2(fl32(dY * gscale)) as [T, O].
 * theta (nullable) receives the uncast fp32 estimator, dense, as [T, O].
 */
void sste_oracle_mvue(const uint16_t *dY, int T, int O, uint64_t seed, uint32_t tensor_id, uint32_t step,
                      uint64_t tg_offset, float gscale, int odt, void *gvals, uint16_t *gmeta, uint8_t *dense_q, float *theta)
{
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < O; ++j) {
        for (int64_t tg = 0; tg < T / 4; ++tg) {
            float a[4];
            for (int i = 0; i < 4; ++i) a[i] = bf16_to_f32(dY[(4 * tg + i) * O + j]);
            uint64_t g = (tg_offset + (uint64_t)tg) * (uint64_t)O + (uint64_t)j;
            uint64_t q = g >> 2;
            uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), tensor_id, step};
            uint32_t rnd[4];
            sste_oracle_philox4x32_10(ctr, key, rnd);
            uint32_t k = rnd[g & 3] >> 8;
            float u = (float)k * 0x1p-24f;
            int q0, q1;
            float v0, v1;
            mvue_group(a, u, &q0, &q1, &v0, &v1);
            if (theta) {
                for (int i = 0; i < 4; ++i) theta[(4 * tg + i) * O + j] = 0.0f;
                theta[(4 * tg + q0) * O + j] = v0;
                theta[(4 * tg + q1) * O + j] = v1;
            }
            if (odt != 0) { v0 = v0 * gscale; v1 = v1 * gscale; }
            store_val(gvals, j * (T / 2) + 2 * tg + 0, v0, odt);
            store_val(gvals, j * (T / 2) + 2 * tg + 1, v1, odt);
            uint16_t nib = (uint16_t)(q0 | (q1 << 2));
            int64_t mi = j * (T / 16) + tg / 4;
            if (tg % 4 == 0) gmeta[mi] = 0;
            gmeta[mi] |= (uint16_t)(nib << (4 * (tg % 4)));
            if (dense_q)
                for (int i = 0; i < 4; ++i)
                    dense_q[(4 * tg + i) * O + j] = f32_to_e5m2(a[i] * gscale);
        }
    }
}

/* --------------------------------------- FP8 per-tensor scaling (Sec. 5.2) */

/* amax of a bf16 tensor (exact, order-free) */
float sste_oracle_amax_bf16(const uint16_t *x, int64_t n)
{
    float m = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        float a = fabsf(bf16_to_f32(x[i]));
        if (a > m) m = a;
    }
    return m;
}

/* q = cast_rn_satfinite(fl32(x * scale)) */
void sste_oracle_quantize_bf16(const uint16_t *x, int64_t n, float scale, int odt, uint8_t *q)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        float v = bf16_to_f32(x[i]) * scale;
        q[i] = (odt == 2) ? f32_to_e4m3(v) : f32_to_e5m2(v);
    }
}

/*
 * H1B-KV reference oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what the H1B-KV hot path computes:
 * 1-bit key sketches (Eq. 2), the normalised Hamming inner product (Eq. 3),
 * 4-bit affine value quantisation (Eq. 4) and softmax(alpha/tau) * V_dequant
 * (Eq. 5).  It exists so that the CUDA library can be checked against
 * something that can be read against the paper by eye.  It shares no code,
 * header, table or helper with the CUDA library, and the product path never
 * calls it: only tests, the smoke check and the bench's cpu-baseline leg do.
 *
 * There is no blocking, packing, fusion or online softmax here.  Bits are one
 * byte each, codes one byte each, softmax is two-pass.  The only parallelism
 * is an OpenMP loop over independent (sequence, KV head) units in the layer
 * driver at the bottom, which does not change any arithmetic.
 *
 * Notation.  The paper writes R in R^{b x d} and s = sign(R v) (Section III,
 * Section IV-A).  Here the sketch width b is called m and the matrix is held
 * transposed, Rt[i][j] = R[j][i], row-major [d][m], so (R v)_j =
 * sum_i v_i * Rt[i][j].
 *
 * Readings of points the paper leaves open:
 *   - sign(0) = +1 (bit 1).
 *   - Eq. 4's scale and zero-point come from the min and max of each group of
 *     G consecutive channels of one value vector: Delta = (max-min)/15 rounded
 *     once (round-to-nearest-even) to IEEE binary16, stored zero = min (exact,
 *     the inputs are binary16).  Codes are computed against the STORED Delta.
 *     G = d is the per-vector scheme of Section IV-B.
 *   - "round" is round-half-to-even.
 *   - Delta16 == 0 gives all-zero codes; codes are clamped to [0, 15].
 *   - alpha_t = (m - 2*Hamming)/m, no 1/sqrt(d), no unbiasing.
 *   - every cached token t in [0, len) is attended; len == 0 gives zeros.
 *   - optional rotary position embedding of the rows that enter Eq. 2 (a
 *     neighbour of the path, not an equation of the paper): half-split pairs,
 *     angles from a caller's table, binary32 arithmetic in a stated order, one
 *     rounding to binary16 (h1bo_rope).
 *
 * Pins (tests, CPU only): the +-1 inner product equals m - 2*Hamming (proof of
 * Prop. 1); bit agreement rate tracks 1 - theta/pi (Eq. 1); round trip error
 * <= Delta/2; T = 1, equal keys, tau -> infinity and tau -> 0 limits; a
 * lossless 16-level grid reduces Eq. 5 to a library softmax @ V; hand-worked
 * tiny cases; the fp16-value variant reduces to a library softmax @ V directly;
 * the rotation against a complex multiplication in fp64, position 0 as the
 * identity, norm preservation and the relative-position property.
 * Parity unpinned (conventions of this build, nothing in the
 * paper fixes them): the min/max rule for Delta and zero, round-half-to-even,
 * and the value of tau.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------ */
/* IEEE binary16 <-> double, written out (no compiler half type is used).    */
/* ------------------------------------------------------------------------ */

/* Exact: every binary16 value is a double. */
double h1bo_half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0) {
        v = ldexp((double)f, -24);                 /* subnormal or zero */
    } else if (e == 31) {
        v = f ? NAN : INFINITY;
    } else {
        v = ldexp((double)(1024 + f), e - 25);     /* (1 + f/1024) * 2^(e-15) */
    }
    return sign ? -v : v;
}

/* One rounding, to nearest, ties to even; overflow goes to infinity. */
uint16_t h1bo_double_to_half_rne(double x)
{
    uint16_t sign = 0;
    if (isnan(x)) return 0x7e00;
    if (signbit(x)) { sign = 0x8000; x = -x; }
    if (isinf(x)) return (uint16_t)(sign | 0x7c00);
    if (x == 0.0) return sign;
    int ex;
    (void)frexp(x, &ex);                           /* x = fr * 2^ex, fr in [0.5,1) */
    int e = ex - 1;                                /* x in [2^e, 2^(e+1)) */
    if (e < -14) e = -14;                          /* subnormal range shares 2^-24 spacing */
    /* spacing of binary16 numbers around x is 2^(e-10) */
    double scaled = ldexp(x, 10 - e);              /* exact: power-of-two scaling */
    double r = nearbyint(scaled);                  /* default mode: ties to even */
    /* r is an integer in [0, 2048] */
    if (r >= 2048.0) { r = 1024.0; e += 1; }
    if (e > 15) return (uint16_t)(sign | 0x7c00);
    long ri = (long)r;
    if (ri < 1024) {
        /* subnormal (only possible when e == -14) */
        return (uint16_t)(sign | (uint16_t)ri);
    }
    return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | (uint16_t)(ri - 1024));
}

/* ------------------------------------------------------------------------ */
/* Rotary position embedding of key or query rows before Eq. 2 (the keys a     */
/* Llama-style model caches are the rotated ones). Not an equation of the      */
/* paper: the rotation is the model's; the convention here is the half-split   */
/* one (channel i pairs with channel i + d/2) with the angles handed in as a   */
/* table, so no transcendental function is evaluated on either side.           */
/*   x      [rows][d]        binary16 bit patterns                              */
/*   table  [n_pos][d/2][2]  float32 (cos, sin) of position p, pair i           */
/*   pos    [rows]           position of each row                               */
/*   out    [rows][d]        binary16: x_i' = x_i c - x_{i+d/2} s,              */
/*                                     x_{i+d/2}' = x_{i+d/2} c + x_i s         */
/* The result is rounded to binary16, and that rounding is a decision every     */
/* later step depends on, so it is taken in one stated precision: each product  */
/* and the sum are rounded to binary32 (no fused multiply-add), then the sum    */
/* is rounded once to binary16, to nearest even.                                */
/* ------------------------------------------------------------------------ */
void h1bo_rope(const uint16_t *x, long rows, int d, const float *table, const int32_t *pos, uint16_t *out)
{
    const int hw = d / 2;
    for (long r = 0; r < rows; ++r) {
        const float *t = table + (size_t)pos[r] * hw * 2;
        for (int i = 0; i < hw; ++i) {
            const float a = (float)h1bo_half_to_double(x[r * d + i]);          /* exact */
            const float b = (float)h1bo_half_to_double(x[r * d + i + hw]);
            const float c = t[2 * i], s = t[2 * i + 1];
            volatile float ac = a * c, bs = b * s, bc = b * c, as = a * s;     /* each rounded to binary32 */
            volatile float lo = ac - bs, hi = bc + as;
            out[r * d + i] = h1bo_double_to_half_rne((double)lo);
            out[r * d + i + hw] = h1bo_double_to_half_rne((double)hi);
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Eq. 2: s = sign(R v), one sketch per row.                                  */
/*   x     [rows][d]  binary16 bit patterns (keys or queries)                 */
/*   Rt    [d][m]     float32 (transposed projection, see header)             */
/*   bits  [rows][m]  out: 1 if (R v)_j >= 0 (s_j = +1), else 0 (s_j = -1)     */
/*   y     [rows][m]  out, optional: the projection itself                    */
/*   a     [rows][m]  out, optional: sum_i |v_i * Rt[i][j]| (boundary margin)  */
/* ------------------------------------------------------------------------ */
void h1bo_sketch(const uint16_t *x, long rows, int d, int m, const float *Rt,
                 uint8_t *bits, double *y, double *a)
{
    for (long r = 0; r < rows; ++r) {
        for (int j = 0; j < m; ++j) {
            double acc = 0.0, mag = 0.0;
            for (int i = 0; i < d; ++i) {
                double term = h1bo_half_to_double(x[r * d + i]) * (double)Rt[(long)i * m + j];
                acc += term;
                mag += fabs(term);
            }
            bits[r * m + j] = (acc >= 0.0) ? 1 : 0;
            if (y) y[r * m + j] = acc;
            if (a) a[r * m + j] = mag;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Eq. 4: v_int4 = round(v / Delta) + z, per group of G channels, with        */
/* Delta = (max - min)/15 -> binary16 and the real zero-point z = -min/Delta  */
/* taken inside the round, i.e. code = round((v - min)/Delta16).              */
/*   v       [rows][d]     binary16                                           */
/*   codes   [rows][d]     out: 0..15                                         */
/*   scale16 [rows][d/G]   out: Delta as binary16 bits                        */
/*   zero16  [rows][d/G]   out: min as binary16 bits                          */
/*   xpre    [rows][d]     out, optional: (v - min)/Delta16 before rounding   */
/*   delta64 [rows][d/G]   out, optional: (max - min)/15 before rounding      */
/* ------------------------------------------------------------------------ */
void h1bo_quantize(const uint16_t *v, long rows, int d, int G,
                   uint8_t *codes, uint16_t *scale16, uint16_t *zero16,
                   double *xpre, double *delta64)
{
    int ng = d / G;
    for (long r = 0; r < rows; ++r) {
        for (int g = 0; g < ng; ++g) {
            const uint16_t *vg = v + r * d + g * G;
            double mn = h1bo_half_to_double(vg[0]);
            double mx = mn;
            uint16_t mn_bits = vg[0];
            for (int c = 1; c < G; ++c) {
                double val = h1bo_half_to_double(vg[c]);
                if (val < mn) { mn = val; mn_bits = vg[c]; }
                if (val > mx) mx = val;
            }
            if (mn == 0.0) mn_bits = 0;            /* one spelling of zero: +0 */
            double delta = (mx - mn) / 15.0;
            uint16_t d16 = h1bo_double_to_half_rne(delta);
            double dq = h1bo_half_to_double(d16);
            scale16[r * ng + g] = d16;
            zero16[r * ng + g] = mn_bits;
            if (delta64) delta64[r * ng + g] = delta;
            for (int c = 0; c < G; ++c) {
                double val = h1bo_half_to_double(vg[c]);
                double xq = 0.0;
                int code = 0;
                if (dq != 0.0) {
                    xq = (val - mn) / dq;
                    double rq = nearbyint(xq);     /* ties to even */
                    if (rq < 0.0) rq = 0.0;
                    if (rq > 15.0) rq = 15.0;
                    code = (int)rq;
                }
                codes[r * d + g * G + c] = (uint8_t)code;
                if (xpre) xpre[r * d + g * G + c] = xq;
            }
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Eq. 3: alpha_t = (1/m) s_t^T s_q, returned as the integer m * alpha_t.     */
/* Computed twice, as the +-1 inner product and as m - 2 * (number of         */
/* disagreeing bits) (proof of Prop. 1); returns how many tokens disagree     */
/* between the two (always 0 unless this file is broken).                     */
/* ------------------------------------------------------------------------ */
long h1bo_scores(const uint8_t *qbits, const uint8_t *kbits, long T, int m,
                 int32_t *score)
{
    long bad = 0;
    for (long t = 0; t < T; ++t) {
        int dot = 0, ham = 0;
        for (int j = 0; j < m; ++j) {
            int sq = qbits[j] ? 1 : -1;
            int sk = kbits[t * m + j] ? 1 : -1;
            dot += sq * sk;
            ham += (qbits[j] != kbits[t * m + j]);
        }
        if (dot != m - 2 * ham) ++bad;
        score[t] = dot;
    }
    return bad;
}

/* ------------------------------------------------------------------------ */
/* Eq. 5: out = softmax(alpha / tau) * V_dequant for one query head.          */
/*   score   [T]          m * alpha_t from h1bo_scores                         */
/*   codes   [T][d], scale16/zero16 [T][d/G]: the cached 4-bit values          */
/*   out     [d]          fp64                                                 */
/*   p       [T]          out, optional: the softmax weights                   */
/* T == 0 gives zeros.                                                         */
/* ------------------------------------------------------------------------ */
void h1bo_attention(const int32_t *score, long T, int m, double inv_tau,
                    const uint8_t *codes, const uint16_t *scale16,
                    const uint16_t *zero16, int d, int G, double *out, double *p)
{
    int ng = d / G;
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    if (T <= 0) return;
    double *w = (double *)malloc(sizeof(double) * (size_t)T);
    double mx = -INFINITY;
    for (long t = 0; t < T; ++t) {
        double alpha = (double)score[t] / (double)m;
        w[t] = alpha * inv_tau;                    /* logit alpha_t / tau */
        if (w[t] > mx) mx = w[t];
    }
    double sum = 0.0;
    for (long t = 0; t < T; ++t) { w[t] = exp(w[t] - mx); sum += w[t]; }
    for (long t = 0; t < T; ++t) {
        double pt = w[t] / sum;
        if (p) p[t] = pt;
        for (int c = 0; c < d; ++c) {
            int g = c / G;
            double vhat = (double)codes[t * d + c] * h1bo_half_to_double(scale16[t * ng + g])
                        + h1bo_half_to_double(zero16[t * ng + g]);
            out[c] += pt * vhat;
        }
    }
    free(w);
}

/* ------------------------------------------------------------------------ */
/* Eq. 5 with uncompressed values: the "1-bit-key only" row of the ablation   */
/* (Table V): out = softmax(alpha / tau) * V, V kept as binary16.              */
/*   score [T] from h1bo_scores, v16 [T][d] binary16, out [d] fp64             */
/* ------------------------------------------------------------------------ */
void h1bo_attention_fp16_values(const int32_t *score, long T, int m, double inv_tau,
                                const uint16_t *v16, int d, double *out)
{
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    if (T <= 0) return;
    double *w = (double *)malloc(sizeof(double) * (size_t)T);
    double mx = -INFINITY, sum = 0.0;
    for (long t = 0; t < T; ++t) {
        w[t] = ((double)score[t] / (double)m) * inv_tau;
        if (w[t] > mx) mx = w[t];
    }
    for (long t = 0; t < T; ++t) { w[t] = exp(w[t] - mx); sum += w[t]; }
    for (long t = 0; t < T; ++t) {
        double pt = w[t] / sum;
        for (int c = 0; c < d; ++c) out[c] += pt * h1bo_half_to_double(v16[t * d + c]);
    }
    free(w);
}

/* Layer driver of the key-only variant: like h1bo_layer, values uncompressed. */
long h1bo_layer_fp16_values(const uint16_t *K, const uint16_t *V, const int32_t *lens,
                            const uint16_t *q, const float *Rt, int B, long T, int Hq,
                            int Hkv, int d, int m, double inv_tau, double *out)
{
    long bad_total = 0;
    int rep = Hq / Hkv;
    long units = (long)B * Hkv;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : bad_total)
#endif
    for (long u = 0; u < units; ++u) {
        int b = (int)(u / Hkv), g = (int)(u % Hkv);
        long len = lens[b];
        size_t n = (size_t)(len > 0 ? len : 1);
        uint16_t *krow = (uint16_t *)malloc(n * d * sizeof(uint16_t));
        uint16_t *vrow = (uint16_t *)malloc(n * d * sizeof(uint16_t));
        uint8_t *kbits = (uint8_t *)malloc(n * m);
        int32_t *score = (int32_t *)malloc(n * sizeof(int32_t));
        uint8_t *qbits = (uint8_t *)malloc((size_t)m);
        for (long t = 0; t < len; ++t) {
            memcpy(krow + t * d, K + (((size_t)b * T + t) * Hkv + g) * d, d * sizeof(uint16_t));
            memcpy(vrow + t * d, V + (((size_t)b * T + t) * Hkv + g) * d, d * sizeof(uint16_t));
        }
        h1bo_sketch(krow, len, d, m, Rt, kbits, NULL, NULL);
        for (int r = 0; r < rep; ++r) {
            int h = g * rep + r;
            h1bo_sketch(q + ((size_t)b * Hq + h) * d, 1, d, m, Rt, qbits, NULL, NULL);
            bad_total += h1bo_scores(qbits, kbits, len, m, score);
            h1bo_attention_fp16_values(score, len, m, inv_tau, vrow, d, out + ((size_t)b * Hq + h) * d);
        }
        free(krow); free(vrow); free(kbits); free(score); free(qbits);
    }
    return bad_total;
}

/* ------------------------------------------------------------------------ */
/* Layer driver: the whole path for one layer, straight from fp16 K/V/q.      */
/*   K, V  [B][T][Hkv][d]  binary16 (T = stride; lens[b] <= T tokens are used)  */
/*   q     [B][Hq][d]      binary16                                            */
/*   Rt    [d][m]          float32                                             */
/*   out   [B][Hq][d]      fp64                                                */
/* Query head h reads KV head h / (Hq/Hkv).  Units (b, kv head) are            */
/* independent and are spread over OpenMP threads; nothing else is parallel.   */
/* Returns the number of score-identity violations (0).                        */
/* ------------------------------------------------------------------------ */
long h1bo_layer(const uint16_t *K, const uint16_t *V, const int32_t *lens,
                const uint16_t *q, const float *Rt, int B, long T, int Hq,
                int Hkv, int d, int m, int G, double inv_tau, double *out)
{
    long bad_total = 0;
    int ng = d / G;
    int rep = Hq / Hkv;
    long units = (long)B * Hkv;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : bad_total)
#endif
    for (long u = 0; u < units; ++u) {
        int b = (int)(u / Hkv), g = (int)(u % Hkv);
        long len = lens[b];
        size_t n = (size_t)(len > 0 ? len : 1);
        uint16_t *krow = (uint16_t *)malloc(n * d * sizeof(uint16_t));
        uint16_t *vrow = (uint16_t *)malloc(n * d * sizeof(uint16_t));
        uint8_t *kbits = (uint8_t *)malloc(n * m);
        uint8_t *codes = (uint8_t *)malloc(n * d);
        uint16_t *sc = (uint16_t *)malloc(n * ng * sizeof(uint16_t));
        uint16_t *zr = (uint16_t *)malloc(n * ng * sizeof(uint16_t));
        int32_t *score = (int32_t *)malloc(n * sizeof(int32_t));
        uint8_t *qbits = (uint8_t *)malloc((size_t)m);
        for (long t = 0; t < len; ++t) {
            memcpy(krow + t * d, K + (((size_t)b * T + t) * Hkv + g) * d, d * sizeof(uint16_t));
            memcpy(vrow + t * d, V + (((size_t)b * T + t) * Hkv + g) * d, d * sizeof(uint16_t));
        }
        h1bo_sketch(krow, len, d, m, Rt, kbits, NULL, NULL);           /* Eq. 2 */
        h1bo_quantize(vrow, len, d, G, codes, sc, zr, NULL, NULL);     /* Eq. 4 */
        for (int r = 0; r < rep; ++r) {
            int h = g * rep + r;
            const uint16_t *qh = q + ((size_t)b * Hq + h) * d;
            h1bo_sketch(qh, 1, d, m, Rt, qbits, NULL, NULL);           /* Eq. 2 on q */
            bad_total += h1bo_scores(qbits, kbits, len, m, score);     /* Eq. 3 */
            h1bo_attention(score, len, m, inv_tau, codes, sc, zr, d, G,
                           out + ((size_t)b * Hq + h) * d, NULL);      /* Eq. 5 */
        }
        free(krow); free(vrow); free(kbits); free(codes);
        free(sc); free(zr); free(score); free(qbits);
    }
    return bad_total;
}

/* ------------------------------------------------------------------------ */
/* Decode step over an existing compressed cache (what one generated token    */
/* costs once the history has been compressed): Eq. 2 on the queries, Eq. 3   */
/* and Eq. 5 against the cached sketches and codes.                           */
/*   kbits  [B][Hkv][T][m] (0/1 bytes), codes [B][Hkv][T][d],                 */
/*   scale16, zero16 [B][Hkv][T][d/G]; T = stride, lens[b] tokens are used    */
/*   q [B][Hq][d] binary16, out [B][Hq][d] fp64                               */
/* OpenMP over the independent (sequence, KV head) units only.                */
/* ------------------------------------------------------------------------ */
long h1bo_decode_cached(const uint8_t *kbits, const uint8_t *codes, const uint16_t *scale16,
                        const uint16_t *zero16, const int32_t *lens, const uint16_t *q,
                        const float *Rt, int B, long T, int Hq, int Hkv, int d, int m, int G,
                        double inv_tau, double *out)
{
    long bad_total = 0;
    int ng = d / G, rep = Hq / Hkv;
    long units = (long)B * Hkv;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : bad_total)
#endif
    for (long u = 0; u < units; ++u) {
        int b = (int)(u / Hkv);
        long len = lens[b];
        int32_t *score = (int32_t *)malloc(sizeof(int32_t) * (size_t)(len > 0 ? len : 1));
        uint8_t *qbits = (uint8_t *)malloc((size_t)m);
        for (int r = 0; r < rep; ++r) {
            int h = (int)(u % Hkv) * rep + r;
            h1bo_sketch(q + ((size_t)b * Hq + h) * d, 1, d, m, Rt, qbits, NULL, NULL);
            bad_total += h1bo_scores(qbits, kbits + (size_t)u * T * m, len, m, score);
            h1bo_attention(score, len, m, inv_tau, codes + (size_t)u * T * d,
                           scale16 + (size_t)u * T * ng, zero16 + (size_t)u * T * ng, d, G,
                           out + ((size_t)b * Hq + h) * d, NULL);
        }
        free(score); free(qbits);
    }
    return bad_total;
}

/* Section IV-B storage statement: a token holds an m-bit sketch and d 4-bit
 * codes; this build also stores a binary16 scale and zero per group. */
long h1bo_entry_bytes(int d, int m, int G)
{
    return (long)m / 8 + (long)d / 2 + (long)(d / G) * 4;
}

/* How many OpenMP threads the layer drivers may use from now on (n < 1: leave it). Changes no arithmetic:
 * the units that the threads share are independent. Returns the previous setting. */
int h1bo_set_threads(int n)
{
#ifdef _OPENMP
    const int before = omp_get_max_threads();
    if (n >= 1) omp_set_num_threads(n);
    return before;
#else
    (void)n;
    return 1;
#endif
}

int h1bo_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * kvq_oracle.c -- plain CPU oracle for the adaptive KV-cache quantization hot
 * path (controller decision -> quantize-append -> decode attention).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is slow on purpose, shares no code
 * with the CUDA library, and may only be called from the tests, from the
 * smoke check and from the benchmark's CPU-baseline leg.  The product path
 * never routes through it.
 *
 * What the paper fixes and what it leaves open:
 *   - Eq. 19-23: three linear layers with two ReLUs, argmax over four logits,
 *     class index -> bit-width {2,4,8,16} (Algorithm 1, label map).
 *   - Eq. 24: the chosen bit-width quantizes both the key row and the value
 *     row of the token before they are appended (Eq. 4).
 *   - Eq. 5: a = Softmax(q K^T / sqrt(d_k)) V over the cached rows.
 *   - The quantizer Q_b itself is only named.  The reading taken here:
 *     per token and per KV head, asymmetric min-max over the head dimension;
 *     scale = (max-min)/(2^b-1) in fp32, stored as fp16; zero-point = the row
 *     minimum (an fp16 input value, -0 stored as +0); codes =
 *     clamp(rint((x-min) * (1/scale_fp16)), 0, 2^b-1), round-half-to-even;
 *     16 "bits" means the fp16 row is stored unchanged.
 *
 * Pins (tests that tie each function to something other than itself):
 *   half<->float   : every fp16 pattern and the halfway cases against numpy.
 *   select_bits    : closed forms (identity weights, zero weights -> class 0),
 *                    fp64 matrix products from numpy away from near-ties,
 *                    argmax(softmax(o)) == argmax(o).
 *   assign_slots   : bijection / counting invariants.
 *   quantize_row   : hand-worked rows (tests/golden), codes in range,
 *                    |x - xhat| <= scale/2, fp16 rows unchanged, min -> 0,
 *                    max -> 2^b-1, grid rows round-trip exactly.
 *   decode_attn    : all-fp16 cache == fp64 softmax attention from a library
 *                    routine; one token -> that token's value row; identical
 *                    keys -> mean of values; convex-hull bound; brute force on
 *                    8-token caches written out term by term in the test.
 *   The paper prints no worked numerical example for any of these steps, so
 *   no pin is a value printed by the paper.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 * (-ffp-contract=off matters: the controller's fp32 multiply and add must each
 * round on their own).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)

/* ------------------------------------------------------------------ fp16 */

/* IEEE binary16 bit pattern -> value.  Written from the format definition:
 * 1 sign, 5 exponent (bias 15), 10 fraction bits. */
float oracle_half_to_float(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24);                 /* subnormal: m * 2^-24 */
    else if (e == 31)
        v = m ? (double)NAN : (double)INFINITY;
    else
        v = ldexp((double)(1024 + m), e - 25);     /* (1 + m/1024) * 2^(e-15) */
    return (float)(sign ? -v : v);
}

/* value -> nearest binary16, ties to even, overflow to infinity. */
static uint16_t double_to_half(double f)
{
    uint16_t sign = signbit(f) ? 0x8000u : 0u;
    double a = fabs(f);
    if (isnan(f))
        return (uint16_t)(sign | 0x7E00u);
    if (a >= 65520.0)                              /* halfway to 2^16 rounds up (even) */
        return (uint16_t)(sign | 0x7C00u);
    if (a == 0.0)
        return sign;
    int ex;
    (void)frexp(a, &ex);                           /* a = frac * 2^ex, frac in [0.5,1) */
    int e = ex - 1;                                /* a in [2^e, 2^(e+1)) */
    if (e < -14)
        e = -14;                                   /* subnormal range shares the 2^-24 step */
    double ulp = ldexp(1.0, e - 10);
    double r = nearbyint(a / ulp);                 /* exact quotient; default mode = ties-to-even */
    if (r >= 2048.0) {                             /* rounded up into the next binade */
        r = 1024.0;
        e += 1;
    }
    int ri = (int)r;
    if (ri < 1024)                                 /* only possible when e == -14: subnormal */
        return (uint16_t)(sign | ri);
    return (uint16_t)(sign | ((e + 15) << 10) | (ri - 1024));
}

uint16_t oracle_float_to_half(float f)
{
    return double_to_half((double)f);              /* float -> double is exact */
}

void oracle_half_to_float_array(const uint16_t *h, int n, float *out)
{
    for (int i = 0; i < n; ++i)
        out[i] = oracle_half_to_float(h[i]);
}

void oracle_float_to_half_array(const float *f, int n, uint16_t *out)
{
    for (int i = 0; i < n; ++i)
        out[i] = oracle_float_to_half(f[i]);
}

/* ------------------------------------------------------------ controller */

static int class_to_bits(int c)
{
    static const int tab[4] = {2, 4, 8, 16};       /* Algorithm 1: {2,4,8,16} <-> {0,1,2,3} */
    return tab[c];
}

static int bits_to_class(int bits)
{
    switch (bits) {
    case 2: return 0;
    case 4: return 1;
    case 8: return 2;
    case 16: return 3;
    default: return -1;
    }
}

/* One linear layer in fp32, Eq. 19-21: out_j = b_j + sum_i W[j][i] * x_i,
 * multiply rounded, then add rounded, i ascending. */
static void linear_f32(const float *W, const float *b, const float *x,
                       int n_out, int n_in, float *out)
{
    for (int j = 0; j < n_out; ++j) {
        float acc = b[j];
        for (int i = 0; i < n_in; ++i) {
            float prod = W[(size_t)j * n_in + i] * x[i];
            acc = acc + prod;
        }
        out[j] = acc;
    }
}

static void relu_f32(float *x, int n)
{
    for (int i = 0; i < n; ++i)
        x[i] = (x[i] > 0.0f) ? x[i] : 0.0f;
}

/* Eq. 19-23 for n tokens.  feats [n][4]; W1 [hidden][4]; W2 [hidden][hidden];
 * W3 [4][hidden].  bits_out [n] in {2,4,8,16}.  logits_out [n][4] and
 * gap_out [n] (largest minus second-largest logit) are optional.
 * Softmax is monotone, so the argmax of Eq. 23 is taken on the logits.
 * Ties go to the lowest class; a NaN logit selects the fp16 class. */
int oracle_select_bits(const float *feats, int n, int hidden,
                       const float *W1, const float *b1,
                       const float *W2, const float *b2,
                       const float *W3, const float *b3,
                       uint8_t *bits_out, float *logits_out, float *gap_out)
{
    if (!feats || !W1 || !b1 || !W2 || !b2 || !W3 || !b3 || !bits_out || n < 0 || hidden < 1)
        return ORACLE_ERR_ARG;
    float *h1 = (float *)malloc(sizeof(float) * (size_t)hidden);
    float *h2 = (float *)malloc(sizeof(float) * (size_t)hidden);
    if (!h1 || !h2) {
        free(h1);
        free(h2);
        return ORACLE_ERR_ARG;
    }
    for (int t = 0; t < n; ++t) {
        float o[4];
        linear_f32(W1, b1, feats + (size_t)t * 4, hidden, 4, h1);
        relu_f32(h1, hidden);
        linear_f32(W2, b2, h1, hidden, hidden, h2);
        relu_f32(h2, hidden);
        linear_f32(W3, b3, h2, 4, hidden, o);

        int cls = 0, has_nan = 0;
        for (int k = 0; k < 4; ++k)
            if (isnan(o[k]))
                has_nan = 1;
        if (has_nan) {
            cls = 3;
        } else {
            for (int k = 1; k < 4; ++k)
                if (o[k] > o[cls])                 /* strict: first maximum wins */
                    cls = k;
        }
        bits_out[t] = (uint8_t)class_to_bits(cls);
        if (logits_out)
            memcpy(logits_out + (size_t)t * 4, o, sizeof(o));
        if (gap_out) {
            float best = -INFINITY, second = -INFINITY;
            for (int k = 0; k < 4; ++k) {
                if (o[k] > best) {
                    second = best;
                    best = o[k];
                } else if (o[k] > second) {
                    second = o[k];
                }
            }
            gap_out[t] = has_nan ? NAN : best - second;
        }
    }
    free(h1);
    free(h2);
    return ORACLE_OK;
}

/* ------------------------------------------------------- slot assignment */

/* Tokens of one (layer, sequence) in position order: pool = class of the
 * token's bit-width; slot = how many earlier tokens of this sequence went to
 * the same pool.  counts[4] carries the pool fill across calls.
 * pool_slot[i] = (pool << 30) | slot. */
int oracle_assign_slots(const uint8_t *bits, int n, uint32_t counts[4], uint32_t *pool_slot)
{
    if (!bits || !counts || !pool_slot || n < 0)
        return ORACLE_ERR_ARG;
    for (int i = 0; i < n; ++i) {
        int p = bits_to_class(bits[i]);
        if (p < 0)
            return ORACLE_ERR_ARG;
        pool_slot[i] = ((uint32_t)p << 30) | counts[p];
        counts[p] += 1;
    }
    return ORACLE_OK;
}

/* -------------------------------------------------------------- quantizer */

/* Row bytes of the packed codes for D elements at this bit-width. */
static int code_bytes(int D, int bits)
{
    return D * bits / 8;
}

/* Q_b of Eq. 24 under the reading in the header comment, for one row of D
 * fp16 values.  codes: D*bits/8 bytes, element i in bits [(i*b)%8, +b) of byte
 * floor(i*b/8); for b == 16 the row's fp16 values, little-endian, unchanged.
 * meta = {scale fp16 bits, zero-point fp16 bits}; {0,0} for b == 16. */
int oracle_quantize_row(const uint16_t *x, int D, int bits, uint8_t *codes, uint16_t meta[2])
{
    if (!x || !codes || !meta || D < 1 || bits_to_class(bits) < 0 || (D * bits) % 8)
        return ORACLE_ERR_ARG;
    if (bits == 16) {
        for (int i = 0; i < D; ++i) {
            codes[2 * i] = (uint8_t)(x[i] & 0xFF);
            codes[2 * i + 1] = (uint8_t)(x[i] >> 8);
        }
        meta[0] = 0;
        meta[1] = 0;
        return ORACLE_OK;
    }
    float mn = oracle_half_to_float(x[0]);
    float mx = mn;
    for (int i = 1; i < D; ++i) {
        float v = oracle_half_to_float(x[i]);
        if (v < mn)
            mn = v;
        if (v > mx)
            mx = v;
    }
    if (mn == 0.0f)
        mn = 0.0f;                                 /* -0 is stored as +0 */
    if (mx == 0.0f)
        mx = 0.0f;                                 /* so that the range of a {-0,+0} row is +0 */
    int levels = (1 << bits) - 1;
    float range = mx - mn;
    float s32 = range / (float)levels;
    uint16_t s16 = oracle_float_to_half(s32);
    float sf = oracle_half_to_float(s16);
    float inv = (sf == 0.0f) ? 0.0f : 1.0f / sf;

    memset(codes, 0, (size_t)code_bytes(D, bits));
    for (int i = 0; i < D; ++i) {
        float v = oracle_half_to_float(x[i]);
        float d = v - mn;
        float scaled = d * inv;
        float r = nearbyintf(scaled);              /* ties-to-even in the default mode */
        if (r < 0.0f)
            r = 0.0f;
        if (r > (float)levels)
            r = (float)levels;
        unsigned c = (unsigned)r;
        int bitpos = i * bits;
        codes[bitpos / 8] |= (uint8_t)(c << (bitpos % 8));
    }
    meta[0] = s16;
    meta[1] = oracle_float_to_half(mn);            /* exact: mn is one of the fp16 inputs */
    return ORACLE_OK;
}

/* xhat_i = float(c_i) * scale + zero_point in fp32 (product rounded, then sum
 * rounded); for b == 16 the stored fp16 value. */
int oracle_dequantize_row(const uint8_t *codes, const uint16_t meta[2], int D, int bits, float *xhat)
{
    if (!codes || !meta || !xhat || D < 1 || bits_to_class(bits) < 0)
        return ORACLE_ERR_ARG;
    if (bits == 16) {
        for (int i = 0; i < D; ++i)
            xhat[i] = oracle_half_to_float((uint16_t)(codes[2 * i] | (codes[2 * i + 1] << 8)));
        return ORACLE_OK;
    }
    float sf = oracle_half_to_float(meta[0]);
    float zp = oracle_half_to_float(meta[1]);
    unsigned mask = (1u << bits) - 1u;
    for (int i = 0; i < D; ++i) {
        int bitpos = i * bits;
        unsigned c = (codes[bitpos / 8] >> (bitpos % 8)) & mask;
        float prod = (float)c * sf;
        xhat[i] = prod + zp;
    }
    return ORACLE_OK;
}

/* Eq. 4 + Eq. 24 for a batch: rows K,V fp16 [batch][n][kv_heads][D], one
 * bit-width per token bits[batch][n] shared by K and V and by every head.
 * Outputs are in position order with a fixed row stride of 2*D bytes:
 * kcodes/vcodes [batch][n][kv_heads][2*D] (unused tail bytes zero),
 * kmeta/vmeta [batch][n][kv_heads][2]. */
int oracle_append(const uint16_t *K, const uint16_t *V, const uint8_t *bits,
                  int batch, int n, int kv_heads, int D,
                  uint8_t *kcodes, uint16_t *kmeta, uint8_t *vcodes, uint16_t *vmeta)
{
    if (!K || !V || !bits || !kcodes || !kmeta || !vcodes || !vmeta)
        return ORACLE_ERR_ARG;
    int bad = 0;
    long rows = (long)batch * n * kv_heads;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (long r = 0; r < rows; ++r) {
        long tok = r / kv_heads;                   /* = b*n + t */
        int b = bits[tok];
        uint8_t *kc = kcodes + (size_t)r * 2 * D;
        uint8_t *vc = vcodes + (size_t)r * 2 * D;
        memset(kc, 0, (size_t)2 * D);
        memset(vc, 0, (size_t)2 * D);
        if (oracle_quantize_row(K + (size_t)r * D, D, b, kc, kmeta + (size_t)r * 2) != ORACLE_OK)
            bad |= 1;
        if (oracle_quantize_row(V + (size_t)r * D, D, b, vc, vmeta + (size_t)r * 2) != ORACLE_OK)
            bad |= 1;
    }
    return bad ? ORACLE_ERR_ARG : ORACLE_OK;
}

/* ------------------------------------------------------- decode attention */

/* Eq. 5 for one query head over n cached tokens of one sequence, all in fp64
 * from the fp32 dequantized rows: logits q.k/sqrt(D), two-pass softmax,
 * weighted sum of value rows.  Rows are read with stride row_stride bytes
 * (codes) and meta_stride uint16 (meta) between consecutive tokens. */
static void attend_one_head(const uint16_t *q, int D, int n, const uint8_t *bits,
                            const uint8_t *kc, const uint16_t *km,
                            const uint8_t *vc, const uint16_t *vm,
                            size_t row_stride, size_t meta_stride,
                            double *out, double *probs)
{
    double *z = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    float *row = (float *)malloc(sizeof(float) * (size_t)D);
    double zmax = -INFINITY;
    double inv_sqrt_d = 1.0 / sqrt((double)D);
    for (int t = 0; t < n; ++t) {
        oracle_dequantize_row(kc + t * row_stride, km + t * meta_stride, D, bits[t], row);
        double dot = 0.0;
        for (int i = 0; i < D; ++i)
            dot += (double)oracle_half_to_float(q[i]) * (double)row[i];
        z[t] = dot * inv_sqrt_d;
        if (z[t] > zmax)
            zmax = z[t];
    }
    double denom = 0.0;
    for (int t = 0; t < n; ++t) {
        z[t] = exp(z[t] - zmax);
        denom += z[t];
    }
    for (int i = 0; i < D; ++i)
        out[i] = 0.0;
    for (int t = 0; t < n; ++t) {
        double p = z[t] / denom;
        if (probs)
            probs[t] = p;
        oracle_dequantize_row(vc + t * row_stride, vm + t * meta_stride, D, bits[t], row);
        for (int i = 0; i < D; ++i)
            out[i] += p * (double)row[i];
    }
    free(z);
    free(row);
}

/* Decode-step attention for a batch.  q [batch][q_heads][D] fp16; the cache is
 * what oracle_append wrote, for n tokens per sequence; query head h reads KV
 * head h / (q_heads/kv_heads).  out [batch][q_heads][D] fp16 (round to nearest
 * even); out64 (optional) the same values before rounding. */
int oracle_decode_attn(const uint16_t *q, int batch, int q_heads, int kv_heads, int D, int n,
                       const uint8_t *bits,
                       const uint8_t *kcodes, const uint16_t *kmeta,
                       const uint8_t *vcodes, const uint16_t *vmeta,
                       uint16_t *out, double *out64)
{
    if (!q || !bits || !kcodes || !kmeta || !vcodes || !vmeta || !out)
        return ORACLE_ERR_ARG;
    if (batch < 1 || q_heads < 1 || kv_heads < 1 || q_heads % kv_heads || n < 1 || D < 1)
        return ORACLE_ERR_ARG;
    int g = q_heads / kv_heads;
    size_t row_stride = (size_t)kv_heads * 2 * D;
    size_t meta_stride = (size_t)kv_heads * 2;
    int units = batch * q_heads;
#pragma omp parallel for schedule(dynamic)
    for (int u = 0; u < units; ++u) {
        int b = u / q_heads, h = u % q_heads, kvh = h / g;
        double *acc = (double *)malloc(sizeof(double) * (size_t)D);
        size_t base = (size_t)b * n * kv_heads + kvh;
        attend_one_head(q + (size_t)u * D, D, n, bits + (size_t)b * n,
                        kcodes + base * 2 * D, kmeta + base * 2,
                        vcodes + base * 2 * D, vmeta + base * 2,
                        row_stride, meta_stride, acc, NULL);
        for (int i = 0; i < D; ++i) {
            out[(size_t)u * D + i] = double_to_half(acc[i]);
            if (out64)
                out64[(size_t)u * D + i] = acc[i];
        }
        free(acc);
    }
    return ORACLE_OK;
}

/* The attention weights of Eq. 5 themselves: probs [batch][q_heads][n] (fp64), same arguments as
 * oracle_decode_attn.  Used for the attention-variance feature of Eq. 16. */
int oracle_decode_probs(const uint16_t *q, int batch, int q_heads, int kv_heads, int D, int n,
                        const uint8_t *bits,
                        const uint8_t *kcodes, const uint16_t *kmeta,
                        const uint8_t *vcodes, const uint16_t *vmeta,
                        double *probs)
{
    if (!q || !bits || !kcodes || !kmeta || !vcodes || !vmeta || !probs)
        return ORACLE_ERR_ARG;
    if (batch < 1 || q_heads < 1 || kv_heads < 1 || q_heads % kv_heads || n < 1 || D < 1)
        return ORACLE_ERR_ARG;
    int g = q_heads / kv_heads;
    size_t row_stride = (size_t)kv_heads * 2 * D;
    size_t meta_stride = (size_t)kv_heads * 2;
    int units = batch * q_heads;
#pragma omp parallel for schedule(dynamic)
    for (int u = 0; u < units; ++u) {
        int b = u / q_heads, h = u % q_heads, kvh = h / g;
        double *acc = (double *)malloc(sizeof(double) * (size_t)D);
        size_t base = (size_t)b * n * kv_heads + kvh;
        attend_one_head(q + (size_t)u * D, D, n, bits + (size_t)b * n,
                        kcodes + base * 2 * D, kmeta + base * 2,
                        vcodes + base * 2 * D, vmeta + base * 2,
                        row_stride, meta_stride, acc, probs + (size_t)u * n);
        free(acc);
    }
    return ORACLE_OK;
}

/* Threads the OpenMP loops above will use (for the benchmark's report). */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

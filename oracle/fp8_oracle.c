/*
 * fp8_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, CPU-only restatement of the FP8 linear layer with per-tensor
 * scaling bias ("Training and inference of large language models using 8-bit
 * floating point", arXiv 2309.17224).  It exists so that the CUDA library can
 * be checked against something written directly from the paper.  It shares no
 * code, header, table or constant generator with the CUDA path and must only
 * be called from tests, from the smoke check and from the benchmark's
 * cpu_baseline / reference legs.
 *
 * Everything is double precision unless the paper fixes the precision.  The
 * only concession to speed is an OpenMP "parallel for" over independent output
 * rows / elements; there is no blocking, fusion or re-association.
 *
 * Parity pins (see tests/test_oracle_*.py): Table 7 closed forms, exhaustive
 * 256-code round trips, nearest-value brute force in numpy, torch's CPU float8
 * casts on the in-range grid, hand-computed biases, exact small-integer GEMMs.
 * Every function below has at least one such pin; none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* Formats (Appendix A, Eq. 4 and Table 7; special values per Appendix B).    */
/* ------------------------------------------------------------------------- */

enum {
    ORC_P_E4 = 0, /* "FP8 E4 (a)": E=4 M=3 bias 8,  max 240,   code 0x80 = NaN/inf     */
    ORC_P_E5 = 1, /* "FP8 E5 (a)": E=5 M=2 bias 16, max 57344, code 0x80 = NaN/inf     */
    ORC_N_E4 = 2, /* "FP8 E4 (b)": E=4 M=3 bias 7,  max 448,   S.1111.111 = NaN        */
    ORC_N_E5 = 3  /* "FP8 E5 (b)": E=5 M=2 bias 15, max 57344, IEEE-style inf and NaN  */
};

typedef struct {
    int E, M, bias;
    int special; /* 0: negative-zero code is the single NaN; 1: all-ones is NaN; 2: IEEE */
} orc_fmt;

static const orc_fmt FMT[4] = {
    {4, 3, 8, 0},
    {5, 2, 16, 0},
    {4, 3, 7, 1},
    {5, 2, 15, 2},
};

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* class of a code: 0 finite, 1 +-inf, 2 NaN */
static int code_class(int f, unsigned code)
{
    const orc_fmt *q = &FMT[f];
    unsigned e = (code >> q->M) & ((1u << q->E) - 1u);
    unsigned m = code & ((1u << q->M) - 1u);
    if (q->special == 0) return code == 0x80u ? 2 : 0;
    if (q->special == 1) return (e == (1u << q->E) - 1u && m == (1u << q->M) - 1u) ? 2 : 0;
    if (e == (1u << q->E) - 1u) return m == 0 ? 1 : 2;
    return 0;
}

/* value = (-1)^sign * 2^(b_exp - bias) * (1 + sum_{i=1..M} d_i 2^-i)   (Eq. 4),
 * with the subnormal rule for b_exp = 0: 2^(1 - bias) * (0 + sum d_i 2^-i). */
double orc_decode(int f, unsigned code)
{
    const orc_fmt *q = &FMT[f];
    code &= 0xFFu;
    int cls = code_class(f, code);
    unsigned s = code >> 7;
    if (cls == 2) return NAN;
    if (cls == 1) return s ? -INFINITY : INFINITY;
    unsigned e = (code >> q->M) & ((1u << q->E) - 1u);
    unsigned m = code & ((1u << q->M) - 1u);
    double frac = (double)m / (double)(1u << q->M);
    double v = (e >= 1) ? ldexp(1.0 + frac, (int)e - q->bias) : ldexp(frac, 1 - q->bias);
    return s ? -v : v;
}

/* Largest finite magnitude of the format ("max_num" of Eq. 3). */
double orc_max_num(int f)
{
    double best = 0.0;
    for (unsigned c = 0; c < 128; ++c)
        if (code_class(f, c) == 0 && orc_decode(f, c) > best) best = orc_decode(f, c);
    return best;
}

/* Round to the nearest representable value, ties to the code with an even
 * last bit; magnitudes beyond the largest finite value are clipped to it and
 * values that round to nothing become zero (Appendix A, the paragraph after
 * Eq. 4).  Done as a search through all finite magnitude codes; the decoded
 * magnitudes are tabulated once per format (orc_decode of codes 0..127). */
static double MAG[4][128];
static int MAG_FINITE[4][128];
static int MAG_READY[4];

static void mag_table(int f)
{
    if (MAG_READY[f]) return;
#pragma omp critical(orc_mag_table)
    {
        if (!MAG_READY[f]) {
            for (unsigned c = 0; c < 128; ++c) {
                MAG_FINITE[f][c] = code_class(f, c) == 0;
                MAG[f][c] = MAG_FINITE[f][c] ? orc_decode(f, c) : 0.0;
            }
#pragma omp flush
            MAG_READY[f] = 1;
        }
    }
}

unsigned orc_encode(int f, double v)
{
    if (isnan(v)) return FMT[f].special == 0 ? 0x80u : 0x7Fu;
    mag_table(f);
    unsigned sign = signbit(v) ? 1u : 0u;
    double a = fabs(v);
    unsigned best = 0;
    double best_d = INFINITY;
    unsigned top = 0;
    double top_v = -1.0;
    for (unsigned c = 0; c < 128; ++c) {
        if (!MAG_FINITE[f][c]) continue;
        double cv = MAG[f][c];
        if (cv > top_v) { top_v = cv; top = c; }
        double d = fabs(cv - a);
        if (d < best_d || (d == best_d && (c & 1u) == 0u)) { best_d = d; best = c; }
    }
    if (a >= top_v) best = top; /* clip (covers +-inf) */
    unsigned out = (sign << 7) | best;
    if (FMT[f].special == 0 && out == 0x80u) out = 0x00u; /* no negative zero in the (a) formats */
    return out;
}

/* ------------------------------------------------------------------------- */
/* 16/32-bit helpers                                                          */
/* ------------------------------------------------------------------------- */

static double bf16_to_double(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* IEEE half (Table 7 row "FP16": E=5, M=10, bias 15) -> double, from the bit fields. */
static double f16_to_double(uint16_t h)
{
    unsigned s = h >> 15, e = (h >> 10) & 0x1Fu, m = h & 0x3FFu;
    double v;
    if (e == 0x1Fu) v = m ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)m / 1024.0, -14);
    else v = ldexp(1.0 + (double)m / 1024.0, (int)e - 15);
    return s ? -v : v;
}

/* Element i of a tensor of the given 16/32-bit type (0 bf16, 1 fp16, 2 fp32) as a double: always exact. */
static double load_elem(const void *x, int dtype, int64_t i)
{
    if (dtype == 0) return bf16_to_double(((const uint16_t *)x)[i]);
    if (dtype == 1) return f16_to_double(((const uint16_t *)x)[i]);
    return (double)((const float *)x)[i];
}

/* float -> bfloat16, round to nearest even (NaN stays NaN, overflow -> inf). */
uint16_t orc_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------------- */
/* amax and scaling bias (Eq. 3)                                              */
/* ------------------------------------------------------------------------- */

/* amax = max(|tensor|).  A NaN anywhere makes the result NaN. */
float orc_amax(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld)
{
    double best = 0.0;
    int saw_nan = 0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            double v = fabs(load_elem(x, dtype, r * ld + c));
            if (isnan(v)) saw_nan = 1;
            else if (v > best) best = v;
        }
    return saw_nan ? NAN : (float)best;
}

/* scaling_bias = floor(log2(max_num / amax)) - margin: the largest integer b
 * with amax * 2^b <= max_num, found by trying integers from the top down
 * (ldexp on a double is exact here, so there is no logarithm to mis-round).
 * amax = 0 and non-finite amax give 0 (the paper leaves both undefined). */
int orc_scaling_bias(float amax, double max_num, int margin)
{
    double a = (double)amax;
    if (!(a > 0.0) || isinf(a)) return 0;
    int b = 400;
    while (ldexp(a, b) > max_num) --b;
    return b - margin;
}

/* ------------------------------------------------------------------------- */
/* scale-and-cast (Eq. 1: adding b to the exponent == multiplying by 2^b)     */
/* ------------------------------------------------------------------------- */

/* y[r, c] = encode_f(x[r, c] * 2^shift); y_t[c, r] is the same code.  Either
 * output may be NULL. */
void orc_cast(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld, int shift, int f, uint8_t *y,
              uint8_t *y_t)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            double v = ldexp(load_elem(x, dtype, r * ld + c), shift);
            uint8_t code = (uint8_t)orc_encode(f, v);
            if (y) y[r * cols + c] = code;
            if (y_t) y_t[c * rows + r] = code;
        }
}

/* ------------------------------------------------------------------------- */
/* FP8 matmuls with unscale (Eq. 2 and Section 2.2)                           */
/* ------------------------------------------------------------------------- */

static void decode_all(int f, const uint8_t *codes, int64_t n, double *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_decode(f, codes[i]);
}

/* One output element: sum_k a[k*sa] * b[k*sb], its absolute-value companion,
 * then the unscale by 2^-(shift_a + shift_b). */
static void dot_unscale(const double *a, int64_t sa, const double *b, int64_t sb, int64_t n,
                        int unshift, double *sum, double *abs_sum)
{
    double s = 0.0, t = 0.0;
    for (int64_t k = 0; k < n; ++k) {
        double p = a[k * sa] * b[k * sb];
        s += p;
        t += fabs(p);
    }
    *sum = ldexp(s, -unshift);
    *abs_sum = ldexp(t, -unshift);
}

static void store_result(double v, double t, int64_t idx, double *out64, float *out32,
                         uint16_t *out_bf16, double *out_abs)
{
    float r = (float)v; /* the "FP32 matmul" result: one rounding of the exact value */
    if (out64) out64[idx] = v;
    if (out32) out32[idx] = r;
    if (out_bf16) out_bf16[idx] = orc_f32_to_bf16(r);
    if (out_abs) out_abs[idx] = t;
}

/* Forward: Y[t, n] = (sum_k X8[t, k] * W8[n, k]) * 2^-(s_x + s_w) + bias_vec[n].
 * x8 is [T, K] in format fx, w8 is [N, K] in format fw.  Any output may be NULL. */
void orc_linear_fwd(const uint8_t *x8, int fx, int s_x, const uint8_t *w8, int fw, int s_w,
                    const double *bias_vec, int64_t T, int64_t K, int64_t N, double *out64,
                    float *out32, uint16_t *out_bf16, double *out_abs)
{
    double *X = malloc(sizeof(double) * (size_t)(T * K));
    double *W = malloc(sizeof(double) * (size_t)(N * K));
    decode_all(fx, x8, T * K, X);
    decode_all(fw, w8, N * K, W);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int64_t n = 0; n < N; ++n) {
            double s, a;
            dot_unscale(X + t * K, 1, W + n * K, 1, K, s_x + s_w, &s, &a);
            if (bias_vec) { s += bias_vec[n]; a += fabs(bias_vec[n]); }
            store_result(s, a, t * N + n, out64, out32, out_bf16, out_abs);
        }
    free(X);
    free(W);
}

/* Input gradient: dX[t, k] = (sum_n dY8[t, n] * W8[n, k]) * 2^-(s_g + s_w). */
void orc_linear_dgrad(const uint8_t *dy8, int fg, int s_g, const uint8_t *w8, int fw, int s_w,
                      int64_t T, int64_t K, int64_t N, double *out64, float *out32,
                      uint16_t *out_bf16, double *out_abs)
{
    double *G = malloc(sizeof(double) * (size_t)(T * N));
    double *W = malloc(sizeof(double) * (size_t)(N * K));
    decode_all(fg, dy8, T * N, G);
    decode_all(fw, w8, N * K, W);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int64_t k = 0; k < K; ++k) {
            double s, a;
            dot_unscale(G + t * N, 1, W + k, K, N, s_g + s_w, &s, &a);
            store_result(s, a, t * K + k, out64, out32, out_bf16, out_abs);
        }
    free(G);
    free(W);
}

/* Weight gradient: dW[n, k] = (sum_t dY8[t, n] * X8[t, k]) * 2^-(s_g + s_x). */
void orc_linear_wgrad(const uint8_t *dy8, int fg, int s_g, const uint8_t *x8, int fx, int s_x,
                      int64_t T, int64_t K, int64_t N, double *out64, float *out32,
                      uint16_t *out_bf16, double *out_abs)
{
    double *G = malloc(sizeof(double) * (size_t)(T * N));
    double *X = malloc(sizeof(double) * (size_t)(T * K));
    decode_all(fg, dy8, T * N, G);
    decode_all(fx, x8, T * K, X);
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            double s, a;
            dot_unscale(G + n, N, X + k, K, T, s_g + s_x, &s, &a);
            store_result(s, a, n * K + k, out64, out32, out_bf16, out_abs);
        }
    free(G);
    free(X);
}

/* The same three definitions evaluated only at listed output positions
 * (row[i], col[i]); used where the full product is too large to finish in
 * seconds.  kind: 0 forward, 1 input gradient, 2 weight gradient; a8/b8 are
 * the two operands in the order of the functions above. */
void orc_linear_samples(int kind, const uint8_t *a8, int fa, int s_a, const uint8_t *b8, int fb,
                        int s_b, const double *bias_vec, int64_t T, int64_t K, int64_t N,
                        const int64_t *row, const int64_t *col, int64_t count, double *out64,
                        float *out32, uint16_t *out_bf16, double *out_abs)
{
    /* Eq. 4 evaluated once per code of each operand's format; the sums below read these values
     * in the same order as the full products above. */
    double va[256], vb[256];
    for (unsigned c = 0; c < 256; ++c) { va[c] = orc_decode(fa, c); vb[c] = orc_decode(fb, c); }
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < count; ++i) {
        int64_t r = row[i], c = col[i];
        double s = 0.0, t = 0.0;
        if (kind == 0) { /* Y[r=t, c=n] */
            for (int64_t k = 0; k < K; ++k) {
                double p = va[a8[r * K + k]] * vb[b8[c * K + k]];
                s += p; t += fabs(p);
            }
        } else if (kind == 1) { /* dX[r=t, c=k] */
            for (int64_t n = 0; n < N; ++n) {
                double p = va[a8[r * N + n]] * vb[b8[n * K + c]];
                s += p; t += fabs(p);
            }
        } else { /* dW[r=n, c=k] */
            for (int64_t tt = 0; tt < T; ++tt) {
                double p = va[a8[tt * N + r]] * vb[b8[tt * K + c]];
                s += p; t += fabs(p);
            }
        }
        s = ldexp(s, -(s_a + s_b));
        t = ldexp(t, -(s_a + s_b));
        if (kind == 0 && bias_vec) { s += bias_vec[c]; t += fabs(bias_vec[c]); }
        store_result(s, t, i, out64, out32, out_bf16, out_abs);
    }
}

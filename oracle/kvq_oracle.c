/*
 * kvq_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the fused KV-cache quantizer and its
 * inverse, written from the paper's definitions so that a reader can check it
 * against the paper by eye.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it.  It shares nothing with the CUDA library: no
 * header, no table, no helper.  The product path never routes through it.
 *
 * What is computed (per head-dim vector x in R^D, D even):
 *
 *   forward  (Sec. 3.1 Eq. 1-2; Sec. 3.2 steps 3-4; Sec. 5.1 item 1; Sec. 7.1)
 *     u = s (.) x                                   sign diagonal on the input
 *     Y_k = D^{-1/2} sum_n u_n e^{-2 pi i k n / D}  unitary DFT, k = 0..D/2
 *     z   = pack(Y)                                 Eq. 2 (sqrt 2 on middle bins)
 *     v_c = lambda_c z_c                            per-channel rescale
 *     a_j = max_{c in group j} |v_c|                per-group abs-max, group = g
 *     sigma_j = fp16(a_j / 7)                       scale = absmax / (2^{b-1}-1), b=4
 *     q_c = clamp(rint(v_c / sigma_j), -7, 7)       round half to even
 *     byte_i = (q_{2i+1} << 4) | (q_{2i} & 0xF)     nibble pack (Sec. 3.2)
 *
 *   inverse  (Sec. 3.1: undo the packing of Eq. 2, inverse real DFT, signs last; Sec. 5.1 item 1 for the clamp)
 *     q -> v^ = q sigma_j -> z^ = v^ / max(lambda_c, 1e-6)
 *     Y^ from z^ by undoing Eq. 2, u = unitary inverse real DFT, x^ = s (.) u
 *
 * The DFT is the naive O(D^2) sum.  The only table is cos/sin(2 pi j / D) for
 * j = 0..D-1, looked up at (k n) mod D; that is the definition, not a fast
 * algorithm.  Vectors are independent; an OpenMP loop over vectors is the only
 * parallelism.
 *
 *   base variants (Sec. 3.2 steps 3-4; Sec. 4.1 "Quantization"): the same path with b = 8 (scale = absmax / 127,
 *     codes in [-127, 127], one two's-complement byte per value) and / or one scale per vector (g = D, "per-token").
 *     The *_b entry points take the bit width b in {4, 8}; the entry points without it are b = 4.
 *
 *   learned rotation at inference (Sec. 5.1 item 2): an orthogonal R in R^{DxD} sits between the transform and
 *     lambda: v = lambda (.) (R z) on the way in, z^ = R^T (v^ / max(lambda, 1e-6)) on the way out.  The *_br entry
 *     points take R row-major in fp64 (NULL = no rotation); training R is not part of this.
 *
 * Readings where the paper is silent (each is listed in the design notes):
 *   - DFT sign convention e^{-2 pi i k n / D}; the imaginary part is packed as
 *     the transform returns it (the usual "rfft" convention).
 *   - Eq. 2 is applied verbatim for any even D (96 and 160 included).
 *   - groups are g consecutive coordinates of the packed order, after lambda.
 *   - scales are stored in fp16 (round to nearest even straight from fp64,
 *     saturating at 65504) and the codes are computed against the STORED scale.
 *   - a group whose stored scale is 0 gets all-zero codes.
 *   - a nibble 0x8 decodes to -8 although the encoder never produces it.
 *   - the sign vector comes from the SplitMix64 mixing function applied to
 *     seed + (n+1) * 0x9E3779B97F4A7C15; the top bit set means -1.
 *
 * Parity status: the transform, the scale rule, the rounding rule and the
 * nibble layout are pinned by closed forms, invariants, a library rfft and
 * brute force (tests/test_oracle_*.py).  The exact integer codes of a given
 * input are "parity unpinned" by any value printed in the paper: the paper
 * prints no worked example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define KVQO_F16 0
#define KVQO_BF16 1

/* ------------------------------------------------------------------ */
/* number formats                                                      */
/* ------------------------------------------------------------------ */

/* IEEE binary16 -> fp64, exact. */
double kvqo_f16_to_f64(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24);               /* zero and subnormals */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp((double)(m + 1024), e - 25);   /* (1 + m/1024) 2^(e-15) */
    return sign ? -v : v;
}

/* fp64 -> IEEE binary16, one rounding, round to nearest even, subnormals kept.
 * saturate != 0: finite overflow gives 65504 instead of infinity (scale rule). */
static uint16_t f64_to_f16_impl(double v, int saturate)
{
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    double a = fabs(v);
    if (isnan(v)) return (uint16_t)(sign | 0x7E00u);
    if (a == 0.0) return sign;
    if (a >= 65520.0)                            /* 65504 + half an ulp: ties go to even = inf */
        return (uint16_t)(sign | (saturate && !isinf(a) ? 0x7BFFu : 0x7C00u));
    int ex;
    (void)frexp(a, &ex);                         /* a = m 2^ex, m in [0.5, 1) */
    int e = ex - 1;                              /* floor(log2 a) */
    if (e < -14) {                               /* subnormal: spacing 2^-24 */
        double q = rint(ldexp(a, 24));
        return (uint16_t)(sign | (uint16_t)q);   /* q == 1024 is the smallest normal */
    }
    double q = rint(ldexp(a, 10 - e));           /* in [1024, 2048] */
    if (q >= 2048.0) { q = 1024.0; e += 1; }
    return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | (uint16_t)((int)q - 1024));
}

uint16_t kvqo_f64_to_f16(double v) { return f64_to_f16_impl(v, 0); }
uint16_t kvqo_f64_to_f16_sat(double v) { return f64_to_f16_impl(v, 1); }

/* bfloat16 -> fp64, exact (bfloat16 is the top half of an IEEE binary32). */
double kvqo_bf16_to_f64(uint16_t b)
{
    uint32_t w = (uint32_t)b << 16;
    float f;
    memcpy(&f, &w, 4);
    return (double)f;
}

/* fp64 -> bfloat16, one rounding, round to nearest even. */
uint16_t kvqo_f64_to_bf16(double v)
{
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    double a = fabs(v);
    if (isnan(v)) return (uint16_t)(sign | 0x7FC0u);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    int ex;
    (void)frexp(a, &ex);
    int e = ex - 1;
    if (e < -126) {                              /* subnormal: spacing 2^-133 */
        double q = rint(ldexp(a, 133));
        return (uint16_t)(sign | (uint16_t)q);
    }
    double q = rint(ldexp(a, 7 - e));            /* in [128, 256] */
    if (q >= 256.0) { q = 128.0; e += 1; }
    if (e > 127) return (uint16_t)(sign | 0x7F80u);
    return (uint16_t)(sign | (uint16_t)((e + 127) << 7) | (uint16_t)((int)q - 128));
}

static double widen(uint16_t raw, int dtype)
{
    return dtype == KVQO_BF16 ? kvqo_bf16_to_f64(raw) : kvqo_f16_to_f64(raw);
}

static uint16_t narrow(double v, int dtype)
{
    return dtype == KVQO_BF16 ? kvqo_f64_to_bf16(v) : kvqo_f64_to_f16(v);
}

/* ------------------------------------------------------------------ */
/* sign diagonal (Sec. 3.1: one +-1 per coordinate, drawn once when    */
/* the plan is made; the generator itself is this build's reading)     */
/* ------------------------------------------------------------------ */

uint64_t kvqo_splitmix64_mix(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

void kvqo_signs(int D, uint64_t seed, int8_t *s)
{
    for (int n = 0; n < D; ++n) {
        uint64_t z = kvqo_splitmix64_mix(seed + (uint64_t)(n + 1) * 0x9E3779B97F4A7C15ULL);
        s[n] = (z >> 63) ? -1 : 1;
    }
}

/* ------------------------------------------------------------------ */
/* SRFT, Eq. 1-2, by the definition                                    */
/* ------------------------------------------------------------------ */

typedef struct {
    int D;
    double *c;   /* cos(2 pi j / D), j = 0..D-1 */
    double *s;   /* sin(2 pi j / D) */
} trig_t;

static int trig_init(trig_t *t, int D)
{
    t->D = D;
    t->c = (double *)malloc(sizeof(double) * (size_t)D);
    t->s = (double *)malloc(sizeof(double) * (size_t)D);
    if (!t->c || !t->s) return -1;
    for (int j = 0; j < D; ++j) {
        double a = 2.0 * M_PI * (double)j / (double)D;
        t->c[j] = cos(a);
        t->s[j] = sin(a);
    }
    return 0;
}

static void trig_free(trig_t *t)
{
    free(t->c);
    free(t->s);
}

/* z = pack(F diag(s) x): Eq. 1 then Eq. 2. */
static void srft_forward_one(const trig_t *t, const int8_t *sg, const double *x, double *z)
{
    const int D = t->D, H = D / 2;
    const double rs = 1.0 / sqrt((double)D);
    for (int k = 0; k <= H; ++k) {
        double re = 0.0, im = 0.0;
        for (int n = 0; n < D; ++n) {
            double u = (double)sg[n] * x[n];
            int j = (int)(((long)k * n) % D);
            re += u * t->c[j];            /* Re e^{-i a} =  cos a */
            im -= u * t->s[j];            /* Im e^{-i a} = -sin a */
        }
        re *= rs;
        im *= rs;
        if (k == 0)
            z[0] = re;
        else if (k == H)
            z[H] = re;
        else {
            z[k] = M_SQRT2 * re;
            z[H + k] = M_SQRT2 * im;
        }
    }
}

/* x = diag(s) F^{-1} unpack(z): undo Eq. 2, unitary inverse real DFT, apply s. */
static void srft_inverse_one(const trig_t *t, const int8_t *sg, const double *z, double *x)
{
    const int D = t->D, H = D / 2;
    const double rs = 1.0 / sqrt((double)D);
    for (int n = 0; n < D; ++n) {
        double acc = z[0] + ((n & 1) ? -z[H] : z[H]);
        for (int k = 1; k < H; ++k) {
            double re = z[k] / M_SQRT2, im = z[H + k] / M_SQRT2;
            int j = (int)(((long)k * n) % D);
            acc += 2.0 * (re * t->c[j] - im * t->s[j]);
        }
        x[n] = (double)sg[n] * acc * rs;
    }
}

int kvqo_srft_forward(int D, const int8_t *sg, const double *x, double *z, int64_t N)
{
    if (D < 2 || (D & 1)) return 1;
    trig_t t;
    if (trig_init(&t, D)) return 2;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r)
        srft_forward_one(&t, sg, x + r * D, z + r * D);
    trig_free(&t);
    return 0;
}

int kvqo_srft_inverse(int D, const int8_t *sg, const double *z, double *x, int64_t N)
{
    if (D < 2 || (D & 1)) return 1;
    trig_t t;
    if (trig_init(&t, D)) return 2;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r)
        srft_inverse_one(&t, sg, z + r * D, x + r * D);
    trig_free(&t);
    return 0;
}

/* ------------------------------------------------------------------ */
/* static lambda calibration (Sec. 7.1: "lambda_d = 1 / per-channel   */
/* max of the SRFT output", taken once over a set of calibration      */
/* vectors).  a_c = max_n |z_{n,c}|, lambda_c = 1 / a_c; a channel    */
/* that is zero on every vector gets lambda_c = 1 (reading: any value */
/* serves, the channel carries nothing).  Inputs are half-precision   */
/* bit patterns widened exactly; the maxima are also returned.        */
/* ------------------------------------------------------------------ */
int kvqo_calibrate_lambda(int D, const int8_t *sg, const uint16_t *x, int dtype, int64_t N, double *lambda, double *amax)
{
    if (D < 2 || (D & 1) || N < 0) return 1;
    trig_t t;
    if (trig_init(&t, D)) return 2;
    for (int c = 0; c < D; ++c) amax[c] = 0.0;
    double *xv = (double *)malloc(sizeof(double) * (size_t)D * 2);
    if (!xv) {
        trig_free(&t);
        return 2;
    }
    double *zv = xv + D;
    for (int64_t r = 0; r < N; ++r) {
        for (int n = 0; n < D; ++n) xv[n] = widen(x[r * D + n], dtype);
        srft_forward_one(&t, sg, xv, zv);
        for (int c = 0; c < D; ++c) {
            double a = fabs(zv[c]);
            if (a > amax[c]) amax[c] = a;
        }
    }
    for (int c = 0; c < D; ++c) lambda[c] = amax[c] > 0.0 ? 1.0 / amax[c] : 1.0;
    free(xv);
    trig_free(&t);
    return 0;
}

/* ------------------------------------------------------------------ */
/* nibble layout (Sec. 3.2: byte = (q[2i+1] << 4) | (q[2i] & 0xF))     */
/* ------------------------------------------------------------------ */

void kvqo_pack_nibbles(const int8_t *q, int64_t n, uint8_t *bytes)
{
    for (int64_t i = 0; i < n / 2; ++i)
        bytes[i] = (uint8_t)((((uint8_t)q[2 * i + 1] & 0xF) << 4) | ((uint8_t)q[2 * i] & 0xF));
}

void kvqo_unpack_nibbles(const uint8_t *bytes, int64_t n, int8_t *q)
{
    for (int64_t i = 0; i < n / 2; ++i) {
        int lo = bytes[i] & 0xF, hi = bytes[i] >> 4;
        q[2 * i] = (int8_t)(lo >= 8 ? lo - 16 : lo);      /* two's-complement nibble */
        q[2 * i + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
}

/* ------------------------------------------------------------------ */
/* quantizer                                                           */
/* ------------------------------------------------------------------ */

/* y = R z (transpose == 0) or y = R^T z (transpose != 0); R row-major [D, D].  Plain sums in index order. */
static void rotate_one(int D, const double *R, int transpose, const double *z, double *y)
{
    for (int i = 0; i < D; ++i) {
        double s = 0.0;
        for (int j = 0; j < D; ++j) s += (transpose ? R[(size_t)j * D + i] : R[(size_t)i * D + j]) * z[j];
        y[i] = s;
    }
}

/* codes of one vector to / from their stored bytes: nibble pairs for b = 4, one two's-complement byte per value for b = 8 */
static void store_codes(const int8_t *q, int D, int bits, uint8_t *dst)
{
    if (bits == 4) kvqo_pack_nibbles(q, D, dst);
    else memcpy(dst, q, (size_t)D);
}

static void load_codes(const uint8_t *src, int D, int bits, int8_t *q)
{
    if (bits == 4) kvqo_unpack_nibbles(src, D, q);
    else memcpy(q, src, (size_t)D);
}

static int64_t lambda_row(int64_t r, int64_t n_lambda, int64_t rows_per_lambda)
{
    return n_lambda == 1 ? 0 : r / rows_per_lambda;
}

static int check_common(int D, int g, int64_t N, int64_t n_lambda, int64_t rows_per_lambda)
{
    if (D < 2 || (D & 1) || g < 2 || (g & 1) || D % g) return 1;
    if (N < 0 || n_lambda < 1) return 1;
    if (n_lambda > 1 && (rows_per_lambda < 1 || (N + rows_per_lambda - 1) / rows_per_lambda > n_lambda))
        return 1;
    return 0;
}

/* steps 4-7 for one vector whose packed transform z is given */
static void quantize_one(int D, int g, int bits, const double *z, const float *lam, int8_t *q, uint16_t *scales,
                         double *v_out)
{
    const double qmax = (double)((1 << (bits - 1)) - 1);   /* 2^{b-1} - 1: 7 or 127 */
    double v[D];
    for (int c = 0; c < D; ++c) v[c] = (double)lam[c] * z[c];
    for (int j = 0; j < D / g; ++j) {
        double a = 0.0;
        for (int c = j * g; c < (j + 1) * g; ++c)
            if (fabs(v[c]) > a) a = fabs(v[c]);
        uint16_t sb = kvqo_f64_to_f16_sat(a / qmax);
        double sigma = kvqo_f16_to_f64(sb);
        scales[j] = sb;
        for (int c = j * g; c < (j + 1) * g; ++c) {
            double t = sigma > 0.0 ? rint(v[c] / sigma) : 0.0;   /* rint: half to even */
            if (t > qmax) t = qmax;
            if (t < -qmax) t = -qmax;
            q[c] = (int8_t)t;
        }
    }
    if (v_out) memcpy(v_out, v, sizeof(double) * (size_t)D);
}

/* Forward path on fp64 input rows.  codes (nullable) receives the unpacked
 * int4 codes [N,D]; v_out (nullable) the rescaled transform lambda (.) z. */
int kvqo_encode_f64_br(int D, int g, int bits, const double *rot, const int8_t *sg, const double *x, int64_t N,
                       const float *lam, int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed, uint16_t *scales,
                       int8_t *codes, double *v_out)
{
    if (check_common(D, g, N, n_lambda, rows_per_lambda) || (bits != 4 && bits != 8)) return 1;
    const int row_bytes = D * bits / 8;
    trig_t t;
    if (trig_init(&t, D)) return 2;
    const int G = D / g;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        double z[D], y[D];
        int8_t q[D];
        srft_forward_one(&t, sg, x + r * D, z);
        if (rot) {
            rotate_one(D, rot, 0, z, y);
            memcpy(z, y, sizeof(double) * (size_t)D);
        }
        quantize_one(D, g, bits, z, lam + lambda_row(r, n_lambda, rows_per_lambda) * D, q, scales + r * G,
                     v_out ? v_out + r * D : NULL);
        store_codes(q, D, bits, packed + r * row_bytes);
        if (codes) memcpy(codes + r * D, q, (size_t)D);
    }
    trig_free(&t);
    return 0;
}

int kvqo_encode_f64_b(int D, int g, int bits, const int8_t *sg, const double *x, int64_t N, const float *lam,
                      int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed, uint16_t *scales,
                      int8_t *codes, double *v_out)
{
    return kvqo_encode_f64_br(D, g, bits, NULL, sg, x, N, lam, n_lambda, rows_per_lambda, packed, scales, codes, v_out);
}

int kvqo_encode_f64(int D, int g, const int8_t *sg, const double *x, int64_t N, const float *lam,
                    int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed, uint16_t *scales,
                    int8_t *codes, double *v_out)
{
    return kvqo_encode_f64_b(D, g, 4, sg, x, N, lam, n_lambda, rows_per_lambda, packed, scales, codes, v_out);
}

/* Forward path on fp16 / bf16 rows: widen exactly, then as above. */
int kvqo_encode_br(int D, int g, int bits, const double *rot, const int8_t *sg, const uint16_t *x, int dtype, int64_t N,
                   const float *lam, int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed,
                   uint16_t *scales, int8_t *codes, double *v_out)
{
    if (check_common(D, g, N, n_lambda, rows_per_lambda) || (bits != 4 && bits != 8)) return 1;
    const int row_bytes = D * bits / 8;
    trig_t t;
    if (trig_init(&t, D)) return 2;
    const int G = D / g;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        double xr[D], z[D];
        int8_t q[D];
        for (int n = 0; n < D; ++n) xr[n] = widen(x[r * D + n], dtype);
        srft_forward_one(&t, sg, xr, z);
        if (rot) {
            rotate_one(D, rot, 0, z, xr);
            memcpy(z, xr, sizeof(double) * (size_t)D);
        }
        quantize_one(D, g, bits, z, lam + lambda_row(r, n_lambda, rows_per_lambda) * D, q, scales + r * G,
                     v_out ? v_out + r * D : NULL);
        store_codes(q, D, bits, packed + r * row_bytes);
        if (codes) memcpy(codes + r * D, q, (size_t)D);
    }
    trig_free(&t);
    return 0;
}

int kvqo_encode_b(int D, int g, int bits, const int8_t *sg, const uint16_t *x, int dtype, int64_t N,
                  const float *lam, int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed,
                  uint16_t *scales, int8_t *codes, double *v_out)
{
    return kvqo_encode_br(D, g, bits, NULL, sg, x, dtype, N, lam, n_lambda, rows_per_lambda, packed, scales, codes, v_out);
}

int kvqo_encode(int D, int g, const int8_t *sg, const uint16_t *x, int dtype, int64_t N,
                const float *lam, int64_t n_lambda, int64_t rows_per_lambda, uint8_t *packed,
                uint16_t *scales, int8_t *codes, double *v_out)
{
    return kvqo_encode_b(D, g, 4, sg, x, dtype, N, lam, n_lambda, rows_per_lambda, packed, scales, codes, v_out);
}

/* Inverse path.  out (nullable) gets x^ rounded to dtype; out_f64 (nullable) the
 * unrounded fp64 reconstruction. */
int kvqo_decode_br(int D, int g, int bits, const double *rot, const int8_t *sg, const uint8_t *packed,
                   const uint16_t *scales, int64_t N, const float *lam, int64_t n_lambda, int64_t rows_per_lambda,
                   uint16_t *out, int dtype, double *out_f64)
{
    if (check_common(D, g, N, n_lambda, rows_per_lambda) || (bits != 4 && bits != 8)) return 1;
    const int row_bytes = D * bits / 8;
    trig_t t;
    if (trig_init(&t, D)) return 2;
    const int G = D / g;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        int8_t q[D];
        double z[D], xr[D];
        const float *l = lam + lambda_row(r, n_lambda, rows_per_lambda) * D;
        load_codes(packed + r * row_bytes, D, bits, q);
        for (int c = 0; c < D; ++c) {
            double sigma = kvqo_f16_to_f64(scales[r * G + c / g]);
            double lc = (double)l[c] > 1e-6 ? (double)l[c] : 1e-6;    /* clamp at 1e-6 */
            z[c] = (double)q[c] * sigma / lc;
        }
        if (rot) {
            rotate_one(D, rot, 1, z, xr);
            memcpy(z, xr, sizeof(double) * (size_t)D);
        }
        srft_inverse_one(&t, sg, z, xr);
        for (int n = 0; n < D; ++n) {
            if (out) out[r * D + n] = narrow(xr[n], dtype);
            if (out_f64) out_f64[r * D + n] = xr[n];
        }
    }
    trig_free(&t);
    return 0;
}

int kvqo_decode_b(int D, int g, int bits, const int8_t *sg, const uint8_t *packed, const uint16_t *scales,
                  int64_t N, const float *lam, int64_t n_lambda, int64_t rows_per_lambda, uint16_t *out,
                  int dtype, double *out_f64)
{
    return kvqo_decode_br(D, g, bits, NULL, sg, packed, scales, N, lam, n_lambda, rows_per_lambda, out, dtype, out_f64);
}

int kvqo_decode(int D, int g, const int8_t *sg, const uint8_t *packed, const uint16_t *scales,
                int64_t N, const float *lam, int64_t n_lambda, int64_t rows_per_lambda, uint16_t *out,
                int dtype, double *out_f64)
{
    return kvqo_decode_b(D, g, 4, sg, packed, scales, N, lam, n_lambda, rows_per_lambda, out, dtype, out_f64);
}

/* Decode-step append: quantize S new vectors (one per stream) and write them to
 * row `pos` of caches laid out [S, T_max, D/2] and [S, T_max, D/g]. */
int kvqo_append(int D, int g, const int8_t *sg, const uint16_t *x_new, int dtype, int64_t S,
                const float *lam, int64_t n_lambda, int64_t streams_per_lambda, uint8_t *packed_cache,
                uint16_t *scales_cache, int64_t T_max, int64_t pos)
{
    if (check_common(D, g, S, n_lambda, streams_per_lambda)) return 1;
    if (T_max < 1 || pos < 0 || pos >= T_max) return 1;
    const int G = D / g;
    uint8_t *pk = (uint8_t *)malloc((size_t)S * (D / 2) + 1);
    uint16_t *sc = (uint16_t *)malloc(sizeof(uint16_t) * ((size_t)S * G + 1));
    if (!pk || !sc) { free(pk); free(sc); return 2; }
    int rc = kvqo_encode(D, g, sg, x_new, dtype, S, lam, n_lambda, streams_per_lambda, pk, sc, NULL, NULL);
    if (!rc)
        for (int64_t i = 0; i < S; ++i) {
            memcpy(packed_cache + (i * T_max + pos) * (D / 2), pk + i * (D / 2), (size_t)(D / 2));
            memcpy(scales_cache + (i * T_max + pos) * G, sc + i * G, sizeof(uint16_t) * (size_t)G);
        }
    free(pk);
    free(sc);
    return rc;
}

int kvqo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

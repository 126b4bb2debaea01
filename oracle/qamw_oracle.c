/*
 * QAM-W weight codec: plain CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
 * of what the codec computes, written from the paper.  Only the test-suite, the
 * smoke check and the benchmark's cpu-baseline / reference arm may build or call
 * it.  It shares no code, header, table or constant generator with the CUDA
 * library and must never be linked into it.
 *
 * Conventions
 *   - W is row-major [d_out, d_in]; w_dtype 0 = IEEE f32, 1 = bf16 (uint16 bits).
 *   - "definition path": every quantity in double, the Hadamard product written
 *     out as the O(b^2) matrix-vector product of Section A.1 (Definition of H_b).
 *   - "canonical f32 path": the same mathematics with a fixed f32 operation
 *     order (see orc_front_row), so that a second implementation can reproduce
 *     the exact bits of the 2-D points that the nearest-codeword decision sees.
 *   - Nearest-codeword search is exhaustive over all K codewords, in double,
 *     lowest index wins exact ties (Section 3.6: the Euclidean-nearest
 *     codeword).
 *
 * Parity pins live in tests/test_oracle_*.py.  Unpinned by the paper (pinned only
 * by this repository's own written specification): the sign-mask generator, the
 * Gaussian sample generator, and the exact trained codeword values.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_NONFINITE (-5)

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Counter-based generators (repository specification; the paper only says     */
/* A fixed sequence derived from one 64-bit seed (Section A.1,                */
/* Definition "Sign mask").                                                   */
/* ------------------------------------------------------------------------- */

/* 64-bit finaliser of the published SplitMix64 generator. */
uint64_t orc_mix64(uint64_t x) {
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ULL;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBULL;
    x ^= x >> 31;
    return x;
}

/* sign_j = -1 if the top bit of mix64(seed + (j+1)*golden) is set, else +1.
 * One sign per input coordinate j, the same for every row. */
void orc_make_signs(uint64_t seed, int d_in, int8_t *out) {
    for (int j = 0; j < d_in; ++j) {
        uint64_t h = orc_mix64(seed + 0x9E3779B97F4A7C15ULL * (uint64_t)(j + 1));
        out[j] = (h >> 63) ? (int8_t)-1 : (int8_t)1;
    }
}

/* Uniform in (0,1) from counter n of stream `seed`: 53 top bits, centred. */
static double orc_uniform(uint64_t seed, uint64_t n) {
    uint64_t h = orc_mix64(orc_mix64(seed ^ 0xD1B54A32D192ED03ULL) + 0x9E3779B97F4A7C15ULL * (n + 1));
    return ((double)(h >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}

/* n samples of the unit circular Gaussian f(x,y) = exp(-(x^2+y^2)/2)/(2 pi)
 * (Section 3.6 equation) by the Box-Muller transform: sample i uses counters
 * 2i and 2i+1.  out holds (x_i, y_i) interleaved. */
void orc_gauss_pairs(uint64_t seed, uint64_t n, double *out) {
    const double two_pi = 6.283185307179586476925286766559;
    for (uint64_t i = 0; i < n; ++i) {
        double u1 = orc_uniform(seed, 2 * i);
        double u2 = orc_uniform(seed, 2 * i + 1);
        double rad = sqrt(-2.0 * log(u1));
        out[2 * i] = rad * cos(two_pi * u2);
        out[2 * i + 1] = rad * sin(two_pi * u2);
    }
}

/* ------------------------------------------------------------------------- */
/* Small host helpers                                                          */
/* ------------------------------------------------------------------------- */

static int is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

static int ilog2(int v) {
    int l = 0;
    while ((1 << l) < v) ++l;
    return l;
}

/* Section 3.3: the largest power of two dividing d_in, capped at 1024
 * (examples printed there: 2048 -> 1024, 5632 -> 512). */
int orc_block_size_rule(int d_in) {
    if (d_in <= 0) return 0;
    int b = 1;
    while (b < 1024 && d_in % (2 * b) == 0) b *= 2;
    return b;
}

/* Section 3.1 step 6 / Section 3.7: B = log2 K bits per pair, rows byte aligned. */
int64_t orc_packed_row_bytes(int d_in, int K) {
    int64_t bits = (int64_t)(d_in / 2) * ilog2(K);
    return (bits + 7) / 8;
}

/* Section 3.7 equation: bpw = B/2 + 16/d_in; Section 3.8: the activation-aware
 * variant adds 16 bits per input channel, i.e. 16/d_out per weight. */
double orc_bpw(int d_out, int d_in, int K, int has_channel_scales) {
    double bpw = 0.5 * ilog2(K) + 16.0 / d_in;
    if (has_channel_scales) bpw += 16.0 / d_out;
    return bpw;
}

/* Section B.2: s_j proportional to r_j^alpha, geometric mean normalised to one,
 * then clamped to [1/16, 16] (no re-normalisation after the clamp).
 * r_j is floored at FLT_MIN before the logarithm.  alpha == 0 gives s == 1. */
void orc_channel_scales(const float *act_rms, int d_in, double alpha, float *s_out) {
    double mean_t = 0.0;
    double *t = (double *)malloc(sizeof(double) * (size_t)d_in);
    for (int j = 0; j < d_in; ++j) {
        double r = (double)act_rms[j];
        if (!(r > (double)FLT_MIN)) r = (double)FLT_MIN;
        t[j] = alpha * log(r);
        mean_t += t[j];
    }
    mean_t /= (double)d_in;
    for (int j = 0; j < d_in; ++j) {
        double s = exp(t[j] - mean_t);
        if (s < 1.0 / 16.0) s = 1.0 / 16.0;
        if (s > 16.0) s = 16.0;
        s_out[j] = (float)s;
    }
    free(t);
}

static float bf16_bits_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* One rounding, double -> bf16, round-to-nearest-even (Section 1: the pipeline
 * dequantises to BF16).  Works on the value, not on an intermediate float. */
uint16_t orc_f64_to_bf16(double v) {
    uint16_t sign = (uint16_t)(signbit(v) ? 0x8000u : 0u);
    double a = fabs(v);
    if (isnan(v)) return (uint16_t)(sign | 0x7FC0u);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    int e;
    (void)frexp(a, &e);          /* a = m * 2^e, m in [0.5, 1) */
    int qexp = e - 8;            /* bf16 keeps 8 significant bits */
    if (qexp < -133) qexp = -133; /* subnormal quantum 2^-133 */
    double q = rint(ldexp(a, -qexp)); /* default rounding mode: ties to even */
    double r = ldexp(q, qexp);
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);
    float f = (float)r; /* exact */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

static double w_at(const void *W, int w_dtype, int64_t idx) {
    if (w_dtype == 0) return (double)((const float *)W)[idx];
    return (double)bf16_bits_to_f32(((const uint16_t *)W)[idx]);
}

/* ------------------------------------------------------------------------- */
/* Rotation (Section 3.3, Section A.1: Definitions and Lemma 1)               */
/* ------------------------------------------------------------------------- */

static int parity(unsigned v) {
    int p = 0;
    while (v) {
        p ^= 1;
        v &= v - 1;
    }
    return p;
}

/* out = b^{-1/2} H_b v with H_b[p][q] = (-1)^{popcount(p & q)}: the closed form
 * of the Sylvester recursion H_{2b} = [[H, H], [H, -H]], H_1 = [1]. */
void orc_hadamard_def(const double *v, int b, double *out) {
    double scale = 1.0 / sqrt((double)b);
    for (int p = 0; p < b; ++p) {
        double acc = 0.0;
        for (int q = 0; q < b; ++q) acc += parity((unsigned)(p & q)) ? -v[q] : v[q];
        out[p] = acc * scale;
    }
}

/* The same matrix built by the recursion itself, row-major b*b, entries +-1.
 * Used by the tests to pin orc_hadamard_def. */
void orc_sylvester_matrix(int b, int8_t *H) {
    H[0] = 1;
    for (int n = 1; n < b; n *= 2) {
        /* H currently n x n with leading dimension b */
        for (int p = 0; p < n; ++p)
            for (int q = 0; q < n; ++q) {
                int8_t h = H[p * b + q];
                H[p * b + (q + n)] = h;
                H[(p + n) * b + q] = h;
                H[(p + n) * b + (q + n)] = (int8_t)-h;
            }
    }
}

/* y = R_fwd u = F S u  (Lemma 1). */
void orc_rotate_fwd(const double *u, const int8_t *signs, int d_in, int b, double *y) {
    double *tmp = (double *)malloc(sizeof(double) * (size_t)b);
    for (int blk = 0; blk < d_in / b; ++blk) {
        for (int q = 0; q < b; ++q) tmp[q] = (double)signs[blk * b + q] * u[blk * b + q];
        orc_hadamard_def(tmp, b, y + blk * b);
    }
    free(tmp);
}

/* u = R_inv y = S F y  (Lemma 1; not the same matrix as R_fwd). */
void orc_rotate_inv(const double *y, const int8_t *signs, int d_in, int b, double *u) {
    for (int blk = 0; blk < d_in / b; ++blk) {
        orc_hadamard_def(y + blk * b, b, u + blk * b);
        for (int q = 0; q < b; ++q) u[blk * b + q] *= (double)signs[blk * b + q];
    }
}

/* Unnormalised in-place butterfly, f32, stages h = 1, 2, 4, ..., b/2; in each
 * stage every pair (j, j+h) with bit h of j clear becomes (a+b, a-b).
 * Each output of a stage is one f32 add or subtract of two stage inputs, so the
 * result does not depend on how the pairs of one stage are scheduled. */
void orc_fwht_f32(float *x, int b) {
    for (int h = 1; h < b; h *= 2)
        for (int j = 0; j < b; ++j)
            if ((j & h) == 0) {
                volatile float a = x[j], c = x[j + h];
                volatile float s = a + c, d = a - c;
                x[j] = s;
                x[j + h] = d;
            }
}

void orc_fwht_f64(double *x, int b) {
    for (int h = 1; h < b; h *= 2)
        for (int j = 0; j < b; ++j)
            if ((j & h) == 0) {
                double a = x[j], c = x[j + h];
                x[j] = a + c;
                x[j + h] = a - c;
            }
}

/* ------------------------------------------------------------------------- */
/* Encoder front half: Section B.2 (W D_s), Section 3.1 steps 1-3.            */
/* ------------------------------------------------------------------------- */

/*
 * One row, canonical f32 path.  Mathematically y = F S (x / ||x||) with
 * x_j = W_j s_j; by linearity the normalisation is applied after the butterfly.
 *   (i)   t_j = f32(s_j) * sign_j          (exact)
 *         x_j = f32( f32(W_j) * t_j )
 *   (ii)  ss  = sum_j (double)x_j * (double)x_j   (j ascending, double)
 *         r   = f32( sqrt(ss) )
 *   (iii) h   = butterfly_f32(x) per block of b   (orc_fwht_f32)
 *   (iv)  c_b = f32( 1 / sqrt((double)b) );  g = f32( c_b / r )  (one f32 division)
 *         y_j = f32(h_j * g)
 *         r == 0  ->  y = 0   (Section 3.1 step 1: a zero row encodes as zeros)
 * Returns ORC_ERR_NONFINITE when r is not finite (y is then unspecified).
 */
int orc_front_row(const void *W_row, int w_dtype, int d_in, int b, const float *chan_scale,
                  const int8_t *signs, float *y_out, float *r_out) {
    double ss = 0.0;
    for (int j = 0; j < d_in; ++j) {
        volatile float w = (float)w_at(W_row, w_dtype, j);
        volatile float t = (chan_scale ? chan_scale[j] : 1.0f) * (float)signs[j];
        volatile float x = w * t;
        y_out[j] = x;
        ss += (double)x * (double)x;
    }
    float r = (float)sqrt(ss);
    *r_out = r;
    if (!isfinite(r)) return ORC_ERR_NONFINITE;
    if (r == 0.0f) {
        for (int j = 0; j < d_in; ++j) y_out[j] = 0.0f;
        return ORC_OK;
    }
    for (int blk = 0; blk < d_in / b; ++blk) orc_fwht_f32(y_out + blk * b, b);
    volatile float cb = (float)(1.0 / sqrt((double)b));
    volatile float g = cb / r;
    for (int j = 0; j < d_in; ++j) {
        volatile float y = y_out[j] * g;
        y_out[j] = y;
    }
    return ORC_OK;
}

/* One row, definition path, everything in double:
 * x = W s, r = ||x||_2, u = x / r, y = F S u with the O(b^2) Hadamard product. */
int orc_front_row_def(const void *W_row, int w_dtype, int d_in, int b, const float *chan_scale,
                      const int8_t *signs, double *y_out, double *r_out) {
    double *u = (double *)malloc(sizeof(double) * (size_t)d_in);
    double ss = 0.0;
    for (int j = 0; j < d_in; ++j) {
        u[j] = w_at(W_row, w_dtype, j) * (chan_scale ? (double)chan_scale[j] : 1.0);
        ss += u[j] * u[j];
    }
    double r = sqrt(ss);
    *r_out = r;
    if (!isfinite(r)) {
        free(u);
        return ORC_ERR_NONFINITE;
    }
    if (r == 0.0) {
        for (int j = 0; j < d_in; ++j) y_out[j] = 0.0;
    } else {
        for (int j = 0; j < d_in; ++j) u[j] /= r;
        orc_rotate_fwd(u, signs, d_in, b, y_out);
    }
    free(u);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Pair-scale calibration (Section 3.4 equation).                             */
/* ------------------------------------------------------------------------- */

/*
 * sigma_k = mean_i |z_k| / sqrt(pi/2) over n = min(d_out, 1024) rows at indices
 * floor(t * d_out / n), t = 0..n-1, rows with zero norm skipped.  |z_k| is the
 * modulus of the un-normalised pair (y_2k, y_2k+1) of the canonical f32 path,
 * taken and averaged in double.  Floor: sigma_k >= 1e-4 / sqrt(d_in); if no row
 * qualifies sigma_k = 1 / sqrt(d_in).
 */
int orc_calibrate(const void *W, int w_dtype, int d_out, int d_in, int64_t w_row_stride, int b,
                  const float *chan_scale, const int8_t *signs, float *sigma_out) {
    if (d_in % 2 || !is_pow2(b) || d_in % b) return ORC_ERR_ARG;
    int n = d_out < 1024 ? d_out : 1024;
    int n_pairs = d_in / 2;
    double *acc = (double *)calloc((size_t)n_pairs, sizeof(double));
    float *y = (float *)malloc(sizeof(float) * (size_t)d_in);
    int used = 0, status = ORC_OK;
    size_t esz = w_dtype == 0 ? 4 : 2;
    for (int t = 0; t < n; ++t) {
        int64_t row = ((int64_t)t * d_out) / n;
        float r;
        int rc = orc_front_row((const char *)W + (size_t)(row * w_row_stride) * esz, w_dtype, d_in, b,
                               chan_scale, signs, y, &r);
        if (rc != ORC_OK) {
            status = rc;
            continue;
        }
        if (r == 0.0f) continue;
        ++used;
        for (int k = 0; k < n_pairs; ++k) {
            double a = (double)y[2 * k], c = (double)y[2 * k + 1];
            acc[k] += sqrt(a * a + c * c);
        }
    }
    double floor_sigma = 1e-4 / sqrt((double)d_in);
    for (int k = 0; k < n_pairs; ++k) {
        double s = used ? (acc[k] / (double)used) / sqrt(1.5707963267948966192313216916398)
                        : 1.0 / sqrt((double)d_in);
        if (s < floor_sigma) s = floor_sigma;
        sigma_out[k] = (float)s;
    }
    free(acc);
    free(y);
    return status;
}

/* ------------------------------------------------------------------------- */
/* Search (Section 3.6) and packing (Section 3.1 step 6).                     */
/* ------------------------------------------------------------------------- */

/* Exhaustive nearest codeword in double; lowest index on exact ties.
 * best/second receive the smallest and second smallest squared distances. */
int orc_nearest(double zx, double zy, const float *codebook, int K, double *best, double *second) {
    int arg = 0;
    double d1 = INFINITY, d2 = INFINITY;
    for (int c = 0; c < K; ++c) {
        double dx = zx - (double)codebook[2 * c];
        double dy = zy - (double)codebook[2 * c + 1];
        double d = dx * dx + dy * dy;
        if (d < d1) {
            d2 = d1;
            d1 = d;
            arg = c;
        } else if (d < d2) {
            d2 = d;
        }
    }
    if (best) *best = d1;
    if (second) *second = d2;
    return arg;
}

/* Index k occupies stream bits [k*B, (k+1)*B); stream bit t is bit (t mod 8) of
 * byte floor(t/8).  Padding bits of the last byte are zero. */
void orc_pack_row(const int32_t *idx, int n_pairs, int B, uint8_t *out, int64_t row_bytes) {
    memset(out, 0, (size_t)row_bytes);
    for (int k = 0; k < n_pairs; ++k)
        for (int t = 0; t < B; ++t)
            if ((idx[k] >> t) & 1) {
                int64_t bit = (int64_t)k * B + t;
                out[bit >> 3] |= (uint8_t)(1u << (bit & 7));
            }
}

void orc_unpack_row(const uint8_t *in, int n_pairs, int B, int32_t *idx) {
    for (int k = 0; k < n_pairs; ++k) {
        int32_t v = 0;
        for (int t = 0; t < B; ++t) {
            int64_t bit = (int64_t)k * B + t;
            if ((in[bit >> 3] >> (bit & 7)) & 1) v |= (1 << t);
        }
        idx[k] = v;
    }
}

/*
 * Full encoder (Section 3.1 steps 1-6 after the channel scaling of Section B.2).
 *   z_k = f32( y_j * q_k ), q_k = f32( 1 / (double)sigma_k ), j in {2k, 2k+1}
 *   idx_k = argmin_c |z_k - c|^2 over all K codewords (double arithmetic on the
 *           f32 values of z and of the codebook)
 * Optional outputs (NULL to skip): z_out [d_out*d_in] f32, idx_out
 * [d_out*d_in/2], d2_best / d2_second [d_out*d_in/2].
 * Rows with a non-finite norm get index 0 everywhere and make the call return
 * ORC_ERR_NONFINITE after all rows are processed.
 */
int orc_encode(const void *W, int w_dtype, int d_out, int d_in, int64_t w_row_stride, int b, int K,
               const float *chan_scale, const int8_t *signs, const float *sigma,
               const float *codebook, uint8_t *packed, int64_t packed_row_stride, float *row_norm,
               float *z_out, int32_t *idx_out, double *d2_best, double *d2_second) {
    if (d_in % 2 || !is_pow2(b) || b < 2 || d_in % b || !is_pow2(K)) return ORC_ERR_ARG;
    int B = ilog2(K);
    int n_pairs = d_in / 2;
    int64_t row_bytes = orc_packed_row_bytes(d_in, K);
    if (packed && packed_row_stride < row_bytes) return ORC_ERR_ARG;
    size_t esz = w_dtype == 0 ? 4 : 2;
    int status = ORC_OK;
#pragma omp parallel
    {
        float *y = (float *)malloc(sizeof(float) * (size_t)d_in);
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_pairs);
#pragma omp for schedule(dynamic, 4)
        for (int i = 0; i < d_out; ++i) {
            float r;
            int rc = orc_front_row((const char *)W + (size_t)((int64_t)i * w_row_stride) * esz, w_dtype,
                                   d_in, b, chan_scale, signs, y, &r);
            row_norm[i] = r;
            if (rc != ORC_OK) {
#pragma omp atomic write
                status = rc;
                for (int j = 0; j < d_in; ++j) y[j] = 0.0f;
            }
            for (int k = 0; k < n_pairs; ++k) {
                volatile float q = (float)(1.0 / (double)sigma[k]);
                volatile float zx = y[2 * k] * q;
                volatile float zy = y[2 * k + 1] * q;
                double d1, d2;
                int a = rc == ORC_OK ? orc_nearest((double)zx, (double)zy, codebook, K, &d1, &d2) : 0;
                if (rc != ORC_OK) d1 = d2 = 0.0;
                idx[k] = a;
                int64_t o = (int64_t)i * n_pairs + k;
                if (z_out) {
                    z_out[2 * o] = zx;
                    z_out[2 * o + 1] = zy;
                }
                if (idx_out) idx_out[o] = a;
                if (d2_best) d2_best[o] = d1;
                if (d2_second) d2_second[o] = d2;
            }
            if (packed) orc_pack_row(idx, n_pairs, B, packed + (size_t)((int64_t)i * packed_row_stride), row_bytes);
        }
        free(y);
        free(idx);
    }
    return status;
}

/*
 * Decoder (Section 3.2; Section B.2 for the final division by s_j), all in
 * double, one rounding to bf16 at the end:
 *   yhat_j = C[idx_k] * sigma_k ; u = S F yhat (definition product) ;
 *   what_j = u_j * r / s_j.
 * what_f64 (optional) receives the unrounded values.
 */
int orc_decode(const uint8_t *packed, int64_t packed_row_stride, const float *row_norm,
               const float *chan_scale, const int8_t *signs, const float *sigma, const float *codebook,
               int K, int b, int d_out, int d_in, uint16_t *what_bf16, double *what_f64) {
    if (d_in % 2 || !is_pow2(b) || b < 2 || d_in % b || !is_pow2(K)) return ORC_ERR_ARG;
    int B = ilog2(K);
    int n_pairs = d_in / 2;
#pragma omp parallel
    {
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_pairs);
        double *yh = (double *)malloc(sizeof(double) * (size_t)d_in);
        double *u = (double *)malloc(sizeof(double) * (size_t)d_in);
#pragma omp for schedule(dynamic, 4)
        for (int i = 0; i < d_out; ++i) {
            orc_unpack_row(packed + (size_t)((int64_t)i * packed_row_stride), n_pairs, B, idx);
            for (int k = 0; k < n_pairs; ++k) {
                yh[2 * k] = (double)codebook[2 * idx[k]] * (double)sigma[k];
                yh[2 * k + 1] = (double)codebook[2 * idx[k] + 1] * (double)sigma[k];
            }
            orc_rotate_inv(yh, signs, d_in, b, u);
            for (int j = 0; j < d_in; ++j) {
                double w = u[j] * (double)row_norm[i];
                if (chan_scale) w /= (double)chan_scale[j];
                int64_t o = (int64_t)i * d_in + j;
                if (what_f64) what_f64[o] = w;
                if (what_bf16) what_bf16[o] = orc_f64_to_bf16(w);
            }
        }
        free(idx);
        free(yh);
        free(u);
    }
    return ORC_OK;
}

/*
 * Distortion sums (Corollary 3 / Corollary 4 / Section B.3 definitions):
 *   out[0] = sum (W - What)^2          out[1] = sum W^2
 *   out[2] = sum r_j^2 (W - What)^2    out[3] = sum r_j^2 W^2   (r_j = act_rms, 1 if NULL)
 * rho_w = sqrt(out0/out1); diagonal-M_x rho_o = sqrt(out2/out3).
 */
int orc_distortion(const void *W, int w_dtype, int64_t w_row_stride, const uint16_t *what_bf16,
                   const float *act_rms, int d_out, int d_in, double *out4) {
    double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    for (int i = 0; i < d_out; ++i)
        for (int j = 0; j < d_in; ++j) {
            double w = w_at(W, w_dtype, (int64_t)i * w_row_stride + j);
            double wh = (double)bf16_bits_to_f32(what_bf16[(int64_t)i * d_in + j]);
            double r2 = act_rms ? (double)act_rms[j] * (double)act_rms[j] : 1.0;
            double e = w - wh;
            s0 += e * e;
            s1 += w * w;
            s2 += r2 * e * e;
            s3 += r2 * w * w;
        }
    out4[0] = s0;
    out4[1] = s1;
    out4[2] = s2;
    out4[3] = s3;
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* 2-D Lloyd-Max codebook (Section 3.6).                                       */
/* ------------------------------------------------------------------------- */

/* One exhaustive assignment pass: assign[i] = nearest codeword of sample i
 * (lowest index on ties); returns the mean squared distance. */
double orc_lloyd_assign(const double *samples, uint64_t n, const double *cb, int K, int32_t *assign) {
    double total = 0.0;
#pragma omp parallel for reduction(+ : total) schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        double zx = samples[2 * i], zy = samples[2 * i + 1];
        double d1 = INFINITY;
        int arg = 0;
        for (int c = 0; c < K; ++c) {
            double dx = zx - cb[2 * c], dy = zy - cb[2 * c + 1];
            double d = dx * dx + dy * dy;
            if (d < d1) {
                d1 = d;
                arg = c;
            }
        }
        if (assign) assign[i] = arg;
        total += d1;
    }
    return total / (double)n;
}

static int cmp_codeword(const void *pa, const void *pb) {
    const double *a = (const double *)pa, *b = (const double *)pb;
    double ra = a[0] * a[0] + a[1] * a[1], rb = b[0] * b[0] + b[1] * b[1];
    if (ra < rb) return -1;
    if (ra > rb) return 1;
    double ta = atan2(a[1], a[0]), tb = atan2(b[1], b[0]);
    return (ta > tb) - (ta < tb);
}

/*
 * Sample-based Lloyd iterations on n unit-circular-Gaussian samples of stream
 * `seed` (orc_gauss_pairs):
 *   init      c_i = sqrt(2) * sample_i, i < K
 *   iterate   D_t = mean squared distance of the nearest-codeword assignment of
 *             the current codebook; stop (keeping the current codebook) when
 *             t > 1 and D_{t-1} - D_t <= rel_tol * D_{t-1}, or after max_iters
 *             centroid updates; otherwise every codeword with a non-empty cell
 *             moves to the mean of its cell (sums in sample order, double), an
 *             empty cell keeps its codeword.
 *   finish    sort by (squared radius, angle), round to f32.
 * mse_out = mean squared distance of the samples to the final f32 codebook;
 * mse_trace (optional, max_iters+1 doubles) receives D_1, D_2, ...
 */
/* The same iteration on a sample array handed in (n pairs of doubles): what a codebook fitted to a
 * matrix's own pairs uses. */
int orc_train_codebook_on(const double *samples, uint64_t n, int K, int max_iters, double rel_tol,
                          float *codebook_out, double *mse_out, int *iters_out, double *mse_trace);

int orc_train_codebook(int K, uint64_t n, uint64_t seed, int max_iters, double rel_tol,
                       float *codebook_out, double *mse_out, int *iters_out, double *mse_trace) {
    if (K < 1 || n < (uint64_t)K || max_iters < 0) return ORC_ERR_ARG;
    double *samples = (double *)malloc(sizeof(double) * 2 * n);
    orc_gauss_pairs(seed, n, samples);
    const int rc = orc_train_codebook_on(samples, n, K, max_iters, rel_tol, codebook_out, mse_out, iters_out, mse_trace);
    free(samples);
    return rc;
}

int orc_train_codebook_on(const double *samples, uint64_t n, int K, int max_iters, double rel_tol,
                          float *codebook_out, double *mse_out, int *iters_out, double *mse_trace) {
    if (!samples || K < 1 || n < (uint64_t)K || max_iters < 0) return ORC_ERR_ARG;
    double *cb = (double *)malloc(sizeof(double) * 2 * (size_t)K);
    double *sum = (double *)malloc(sizeof(double) * 2 * (size_t)K);
    int64_t *cnt = (int64_t *)malloc(sizeof(int64_t) * (size_t)K);
    int32_t *assign = (int32_t *)malloc(sizeof(int32_t) * n);
    const double root2 = 1.4142135623730950488016887242097;
    for (int c = 0; c < 2 * K; ++c) cb[c] = root2 * samples[c];
    double prev = INFINITY;
    int updates = 0, t = 0;
    for (;;) {
        double D = orc_lloyd_assign(samples, n, cb, K, assign);
        if (mse_trace) mse_trace[t] = D;
        ++t;
        if (t > 1 && prev - D <= rel_tol * prev) break;
        if (updates >= max_iters) break;
        memset(sum, 0, sizeof(double) * 2 * (size_t)K);
        memset(cnt, 0, sizeof(int64_t) * (size_t)K);
        for (uint64_t i = 0; i < n; ++i) {
            sum[2 * assign[i]] += samples[2 * i];
            sum[2 * assign[i] + 1] += samples[2 * i + 1];
            cnt[assign[i]]++;
        }
        for (int c = 0; c < K; ++c)
            if (cnt[c] > 0) {
                cb[2 * c] = sum[2 * c] / (double)cnt[c];
                cb[2 * c + 1] = sum[2 * c + 1] / (double)cnt[c];
            }
        ++updates;
        prev = D;
    }
    qsort(cb, (size_t)K, 2 * sizeof(double), cmp_codeword);
    for (int c = 0; c < 2 * K; ++c) codebook_out[c] = (float)cb[c];
    if (mse_out) {
        for (int c = 0; c < 2 * K; ++c) cb[c] = (double)codebook_out[c];
        *mse_out = orc_lloyd_assign(samples, n, cb, K, NULL);
    }
    if (iters_out) *iters_out = updates;
    free(cb);
    free(sum);
    free(cnt);
    free(assign);
    return ORC_OK;
}

/* Mean squared distance of n samples of stream `seed` to an f32 codebook. */
double orc_codebook_mse(const float *codebook, int K, uint64_t n, uint64_t seed) {
    double *samples = (double *)malloc(sizeof(double) * 2 * n);
    double *cb = (double *)malloc(sizeof(double) * 2 * (size_t)K);
    orc_gauss_pairs(seed, n, samples);
    for (int c = 0; c < 2 * K; ++c) cb[c] = (double)codebook[c];
    double D = orc_lloyd_assign(samples, n, cb, K, NULL);
    free(samples);
    free(cb);
    return D;
}

/* ------------------------------------------------------------------------- */
/* Polar baseline (Section 3.5; Corollary "Rayleigh-Lloyd polar distortion     */
/* bound" and the Remark after it).                                           */
/* ------------------------------------------------------------------------- */

/* Composite Simpson rule for the three moments of the unit Rayleigh density
 * f(r) = r exp(-r^2/2) on [a, b]: m[q] = int r^q f(r) dr, q = 0, 1, 2. */
static void rayleigh_moments(double a, double b, int n_sub, double m[3]) {
    m[0] = m[1] = m[2] = 0.0;
    if (!(b > a)) return;
    if (n_sub % 2) ++n_sub;
    double h = (b - a) / n_sub;
    for (int i = 0; i <= n_sub; ++i) {
        double r = a + h * i;
        double w = (i == 0 || i == n_sub) ? 1.0 : ((i % 2) ? 4.0 : 2.0);
        double f = r * exp(-0.5 * r * r) * w;
        m[0] += f;
        m[1] += f * r;
        m[2] += f * r * r;
    }
    m[0] *= h / 3.0;
    m[1] *= h / 3.0;
    m[2] *= h / 3.0;
}

#define ORC_RAYLEIGH_RMAX 8.0 /* integration cut-off named in the Remark */

/* Distortion int_0^Rmax (r - Q(r))^2 f(r) dr of the nearest-level quantiser with
 * the given levels (ascending), cells bounded by the midpoints. */
double orc_rayleigh_distortion(const double *levels, int n) {
    double D = 0.0;
    for (int j = 0; j < n; ++j) {
        double lo = j == 0 ? 0.0 : 0.5 * (levels[j - 1] + levels[j]);
        double hi = j == n - 1 ? ORC_RAYLEIGH_RMAX : 0.5 * (levels[j] + levels[j + 1]);
        double m[3];
        rayleigh_moments(lo, hi, 4096, m);
        D += m[2] - 2.0 * levels[j] * m[1] + levels[j] * levels[j] * m[0];
    }
    return D;
}

/* N-level Lloyd-Max quantiser of the unit Rayleigh density under squared error:
 * start from the quantiles r_j = sqrt(-2 ln(1 - (j + 1/2)/N)), then alternate
 * cell boundaries at the midpoints of the levels, every level at the centroid of its cell
 * (numerically integrated on [0, 8]) until no level moves by more than 1e-13 or
 * max_iters rounds.  levels_out: f32 (the practical codebook); returns the
 * numerically integrated distortion C_LM of those f32 levels. */
double orc_rayleigh_lloyd_max(int n, int max_iters, float *levels_out) {
    double *l = (double *)malloc(sizeof(double) * (size_t)n);
    for (int j = 0; j < n; ++j) l[j] = sqrt(-2.0 * log(1.0 - ((double)j + 0.5) / (double)n));
    for (int it = 0; it < max_iters; ++it) {
        double move = 0.0, prev_level = 0.0, next;
        for (int j = 0; j < n; ++j) {
            double lo = j == 0 ? 0.0 : 0.5 * (prev_level + l[j]);
            double hi = j == n - 1 ? ORC_RAYLEIGH_RMAX : 0.5 * (l[j] + l[j + 1]);
            double m[3];
            rayleigh_moments(lo, hi, 4096, m);
            next = m[0] > 0.0 ? m[1] / m[0] : l[j];
            prev_level = l[j]; /* boundaries of this round use the levels of the previous round */
            if (fabs(next - l[j]) > move) move = fabs(next - l[j]);
            l[j] = next;
        }
        if (move < 1e-13) break;
    }
    for (int j = 0; j < n; ++j) {
        levels_out[j] = (float)l[j];
        l[j] = (double)levels_out[j];
    }
    double D = orc_rayleigh_distortion(l, n);
    free(l);
    return D;
}

/* The K = 2^(Ba+Bp) reconstruction points of the polar codec as one table:
 * index = (p << Ba) | a, point = level_a (cos phi_p, sin phi_p) with the bin
 * centres phi_p = (2p + 1) pi / N_p of the Corollary, rounded to f32. */
void orc_polar_codebook(const float *levels, int Ba, int Bp, float *codebook_out) {
    const double pi = 3.14159265358979323846264338327950288;
    int Na = 1 << Ba, Np = 1 << Bp;
    for (int p = 0; p < Np; ++p) {
        double phi = (2.0 * p + 1.0) * pi / (double)Np;
        for (int a = 0; a < Na; ++a) {
            int idx = (p << Ba) | a;
            codebook_out[2 * idx] = (float)((double)levels[a] * cos(phi));
            codebook_out[2 * idx + 1] = (float)((double)levels[a] * sin(phi));
        }
    }
}

/* Polar quantiser of one point: amplitude to the nearest level (lowest index on
 * ties), phase theta in [0, 2 pi) to the bin floor(theta / (2 pi / N_p)); the
 * origin goes to bin 0.  margin_a: (gap between the distances to the two
 * nearest levels) / amplitude; margin_p: distance in radians to the nearest
 * bin boundary (pi when there is one bin or the point is the origin). */
int orc_polar_quantize(double zx, double zy, const float *levels, int Ba, int Bp, double *margin_a,
                       double *margin_p) {
    const double pi = 3.14159265358979323846264338327950288;
    int Na = 1 << Ba, Np = 1 << Bp;
    double r = sqrt(zx * zx + zy * zy);
    int a = 0;
    double d1 = INFINITY, d2 = INFINITY;
    for (int j = 0; j < Na; ++j) {
        double d = fabs(r - (double)levels[j]);
        if (d < d1) {
            d2 = d1;
            d1 = d;
            a = j;
        } else if (d < d2) {
            d2 = d;
        }
    }
    if (margin_a) *margin_a = Na > 1 ? (d2 - d1) / (r > 1e-300 ? r : 1e-300) : INFINITY;
    int p = 0;
    double mp = pi;
    if (Np > 1 && !(zx == 0.0 && zy == 0.0)) {
        double theta = atan2(zy, zx);
        if (theta < 0.0) theta += 2.0 * pi;
        double width = 2.0 * pi / (double)Np;
        p = (int)floor(theta / width);
        if (p >= Np) p = Np - 1;
        double lo = theta - width * p, hi = width * (p + 1) - theta;
        mp = lo < hi ? lo : hi;
    }
    if (margin_p) *margin_p = mp;
    return (p << Ba) | a;
}

/* Encoder with the polar quantiser in place of the nearest-codeword search:
 * everything up to z_k as in orc_encode, then idx_k = orc_polar_quantize(z_k).
 * Optional outputs as in orc_encode, with the two margins in place of the two
 * distances. */
int orc_encode_polar(const void *W, int w_dtype, int d_out, int d_in, int64_t w_row_stride, int b,
                     int Ba, int Bp, const float *chan_scale, const int8_t *signs, const float *sigma,
                     const float *levels, uint8_t *packed, int64_t packed_row_stride, float *row_norm,
                     float *z_out, int32_t *idx_out, double *margin_a, double *margin_p) {
    if (d_in % 2 || !is_pow2(b) || b < 2 || d_in % b || Ba < 0 || Bp < 0 || Ba + Bp < 1) return ORC_ERR_ARG;
    int B = Ba + Bp;
    int n_pairs = d_in / 2;
    int64_t row_bytes = orc_packed_row_bytes(d_in, 1 << B);
    if (packed && packed_row_stride < row_bytes) return ORC_ERR_ARG;
    size_t esz = w_dtype == 0 ? 4 : 2;
    int status = ORC_OK;
#pragma omp parallel
    {
        float *y = (float *)malloc(sizeof(float) * (size_t)d_in);
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_pairs);
#pragma omp for schedule(dynamic, 4)
        for (int i = 0; i < d_out; ++i) {
            float r;
            int rc = orc_front_row((const char *)W + (size_t)((int64_t)i * w_row_stride) * esz, w_dtype,
                                   d_in, b, chan_scale, signs, y, &r);
            row_norm[i] = r;
            if (rc != ORC_OK) {
#pragma omp atomic write
                status = rc;
                for (int j = 0; j < d_in; ++j) y[j] = 0.0f;
            }
            for (int k = 0; k < n_pairs; ++k) {
                volatile float q = (float)(1.0 / (double)sigma[k]);
                volatile float zx = y[2 * k] * q;
                volatile float zy = y[2 * k + 1] * q;
                double ma = INFINITY, mp = INFINITY;
                int a = rc == ORC_OK ? orc_polar_quantize((double)zx, (double)zy, levels, Ba, Bp, &ma, &mp) : 0;
                idx[k] = a;
                int64_t o = (int64_t)i * n_pairs + k;
                if (z_out) {
                    z_out[2 * o] = zx;
                    z_out[2 * o + 1] = zy;
                }
                if (idx_out) idx_out[o] = a;
                if (margin_a) margin_a[o] = ma;
                if (margin_p) margin_p[o] = mp;
            }
            if (packed) orc_pack_row(idx, n_pairs, B, packed + (size_t)((int64_t)i * packed_row_stride), row_bytes);
        }
        free(y);
        free(idx);
    }
    return status;
}

/* ------------------------------------------------------------------------- */
/* Variants around the path.                                                   */
/* ------------------------------------------------------------------------- */

/* Section 3.2: the row norm serialised as binary16 -- metadata rounded to IEEE
 * binary16 (nearest even; overflow to infinity, gradual underflow) and widened
 * back to f32, in place. */
void orc_round_f16(float *v, int64_t n) {
    for (int64_t i = 0; i < n; ++i) {
        double x = (double)v[i];
        if (x != x || x == INFINITY || x == -INFINITY || x == 0.0) continue;
        double a = fabs(x);
        int e;
        frexp(a, &e); /* a = m 2^e, m in [0.5, 1) */
        int q = e - 11; /* spacing 2^q: 11 significant bits */
        if (q < -24) q = -24; /* subnormal spacing 2^-24 */
        double r = nearbyint(ldexp(a, -q)); /* ties to even in the default rounding mode */
        double y = ldexp(r, q);
        if (y >= 65520.0) y = INFINITY; /* beyond the largest finite half (65504) after rounding */
        v[i] = (float)(x < 0 ? -y : y);
    }
}

/* Section A.3, optional final direction renormalisation: the decoder divides the
 * reconstructed direction by its own length before multiplying by the stored row
 * norm.  The rotation preserves lengths (Lemma 1), so that length is
 * |yhat| = sqrt(sum_k sigma_k^2 |c_idx_k|^2); out[i] = f32(r_i / |yhat_i|) is the
 * factor to hand to the decoder in place of r_i (0 for an all-zero yhat). */
int orc_renorm_row_norms(const uint8_t *packed, int64_t packed_row_stride, const float *row_norm,
                         const float *sigma, const float *codebook, int K, int d_out, int d_in, float *out) {
    if (d_in % 2 || !is_pow2(K)) return ORC_ERR_ARG;
    int B = ilog2(K), n_pairs = d_in / 2;
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_pairs);
    for (int i = 0; i < d_out; ++i) {
        orc_unpack_row(packed + (size_t)((int64_t)i * packed_row_stride), n_pairs, B, idx);
        double ss = 0.0;
        for (int k = 0; k < n_pairs; ++k) {
            double cx = (double)codebook[2 * idx[k]] * (double)sigma[k];
            double cy = (double)codebook[2 * idx[k] + 1] * (double)sigma[k];
            ss += cx * cx + cy * cy;
        }
        out[i] = ss > 0.0 ? (float)((double)row_norm[i] / sqrt(ss)) : 0.0f;
    }
    free(idx);
    return ORC_OK;
}

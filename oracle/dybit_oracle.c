/*
 * DyBit CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, obviously-correct restatement of what the DyBit hot path
 * computes: decode (Eq. 1 / Table I), nearest-value encode, per-tensor
 * max-abs scale, dense bit packing, matrix multiply on coded operands and
 * direct convolution on coded operands.  Everything is written the long way
 * (table enumeration, brute-force search, triple / seven-fold loops, exact
 * int64 accumulation); nothing here is blocked, fused or reordered.
 *
 * Only the tests, the smoke check and the bench's CPU-baseline leg may use
 * this file.  It shares no code, header, table or constant with the CUDA
 * library.  OpenMP pragmas only spread independent outer iterations over
 * host cores for the timed baseline; they change no result.
 *
 * Parity pins (tests/test_oracle_*.py): Table I, the Section III-B.2 worked
 * example, monotonicity / distinctness over all 2^N codes, idempotence,
 * numpy/torch fp64 library routines for GEMM and conv.  No function in this
 * file is "parity unpinned".
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* Format helpers                                                      */
/* ------------------------------------------------------------------ */

/* Number of magnitude bits m of a format: a signed N-bit code is one sign
 * bit (the MSB) followed by an unsigned (N-1)-bit DyBit magnitude; an
 * unsigned N-bit code is the magnitude alone (Table I is the unsigned
 * 4-bit case, m = 4). */
static int mag_bits(int bits, int is_signed) { return is_signed ? bits - 1 : bits; }

int orc_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* Decode: Eq. 1, Section III-A                                        */
/* ------------------------------------------------------------------ */

/* Value of the m-bit unsigned magnitude pattern c (0 <= c < 2^m).
 *   c == 0                      -> 0                     (Eq. 1, first case)
 *   start bit 0                 -> the low m-1 bits read as a pure fraction,
 *                                  c / 2^(m-1), inside (0,1)   (Section III-A)
 *   start bit 1                 -> i = number of leading ones before the
 *                                  next zero; after that zero come k
 *                                  fraction bits holding x:
 *                                  2^(i-1) * (1 + x / 2^k)     (Eq. 1, third case)
 *   all ones (i == m, no zero)  -> the largest value.  Table I lists 1111
 *                                  as 8 = 2^(m-1), i.e. the third case with
 *                                  k = 0, x = 0; that reading is used
 *                                  (Eq. 1, second case). */
double orc_decode_mag(int m, unsigned c)
{
    if (c == 0) return 0.0;
    unsigned msb = (c >> (m - 1)) & 1u;
    if (!msb) return (double)c / (double)(1u << (m - 1));
    int i = 0;
    for (int b = m - 1; b >= 0; --b) {
        if ((c >> b) & 1u) ++i; else break;
    }
    if (i == m) return ldexp(1.0, m - 1);
    int k = m - 1 - i;                 /* bits left after the run and its terminating zero */
    unsigned x = c & ((1u << k) - 1u);
    return ldexp(1.0, i - 1) * (1.0 + (double)x / (double)(1u << k));
}

/* Value of a whole code: (-1)^s * magnitude value (Eq. 1).  The pattern
 * "sign set, magnitude zero" decodes to 0. */
double orc_decode(int bits, int is_signed, unsigned code)
{
    int m = mag_bits(bits, is_signed);
    unsigned mag = code & ((1u << m) - 1u);
    double v = orc_decode_mag(m, mag);
    if (is_signed && ((code >> m) & 1u) && v != 0.0) v = -v;
    return v;
}

void orc_decode_table(int bits, int is_signed, double *table /* 2^bits */)
{
    for (unsigned c = 0; c < (1u << bits); ++c) table[c] = orc_decode(bits, is_signed, c);
}

/* The decoder's two output fields (Section III-B.2): exponent = length of
 * the leading-ones run minus one; mantissa = the pattern left-shifted past
 * the run and its terminating zero with the hidden one placed in the MSB of
 * an m-bit word.  Only defined for start bit 1. */
void orc_decode_fields(int m, unsigned c, int *exponent, unsigned *mantissa)
{
    int i = 0;
    for (int b = m - 1; b >= 0; --b) {
        if ((c >> b) & 1u) ++i; else break;
    }
    *exponent = i - 1;
    if (i >= m) { *mantissa = 1u << (m - 1); return; }
    int k = m - 1 - i;
    unsigned x = c & ((1u << k) - 1u);
    /* hidden one at bit m-1, fraction bits directly below it */
    *mantissa = (1u << (m - 1)) | (x << (m - 1 - k));
}

/* ------------------------------------------------------------------ */
/* Scale: per-tensor max-abs (Section I, "precision at the tensor level") */
/* ------------------------------------------------------------------ */

/* amax = largest finite |x|.  scale maps the all-ones code to amax:
 * scale = amax / 2^(m-1); inv = 2^(m-1) / amax, one fp32 division.
 * An all-zero (or empty, or all non-finite) tensor gets scale = inv = 1. */
void orc_absmax_scale(const float *x, int64_t n, int bits, int is_signed,
                      float *scale, float *inv)
{
    int m = mag_bits(bits, is_signed);
    float amax = 0.0f;
    for (int64_t i = 0; i < n; ++i) {
        float a = fabsf(x[i]);
        if (isfinite(a) && a > amax) amax = a;
    }
    if (amax == 0.0f) { *scale = 1.0f; *inv = 1.0f; return; }
    float vmax = ldexpf(1.0f, m - 1);
    *scale = amax / vmax;
    *inv = vmax / amax;
}

/* ------------------------------------------------------------------ */
/* Encode: inverse of Eq. 1 by exhaustive search                       */
/* ------------------------------------------------------------------ */

/* One element.  t = |x| * inv in fp32 (one IEEE multiply); the magnitude
 * code is the c whose value is nearest to t, distances taken exactly in
 * double; of two equally near codes the even one wins; t above the largest
 * value, or infinite, gives the all-ones code; NaN gives code 0.  The sign
 * bit is the sign of x unless the magnitude code is 0.  An unsigned format
 * has no sign bit: a negative x takes the nearest value it has, 0. */
unsigned orc_encode_one(float x, float inv, int bits, int is_signed)
{
    int m = mag_bits(bits, is_signed);
    unsigned ncodes = 1u << m;
    float t = fabsf(x) * inv;
    unsigned best = 0;
    if (isnan(t)) {
        best = 0;
    } else if (isinf(t) || (double)t >= orc_decode_mag(m, ncodes - 1u)) {
        /* at or beyond the largest value: the nearest value is the largest one.
         * (Taken explicitly because for huge t the distances below would all
         * round to the same double.) */
        best = ncodes - 1u;
    } else {
        double bestd = INFINITY;
        for (unsigned c = 0; c < ncodes; ++c) {
            double d = fabs((double)t - orc_decode_mag(m, c));
            if (d < bestd || (d == bestd && (c & 1u) == 0u && (best & 1u) != 0u)) {
                bestd = d;
                best = c;
            }
        }
    }
    unsigned s = 0;
    if (is_signed && best != 0 && signbit(x)) s = 1;
    if (!is_signed && signbit(x)) best = 0;
    return (s << m) | best;
}

/* codes[i] in one byte each (unpacked). */
void orc_quantize(const float *x, int64_t n, int bits, int is_signed, float inv,
                  uint8_t *codes)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        codes[i] = (uint8_t)orc_encode_one(x[i], inv, bits, is_signed);
}

/* ------------------------------------------------------------------ */
/* Pack / unpack: dense little-endian bit stream                       */
/* ------------------------------------------------------------------ */

/* Code j occupies stream bits [j*bits, (j+1)*bits); stream bit b is bit
 * (b % 8) of byte (b / 8).  out must hold out_bytes >= ceil(n*bits/8)
 * bytes; it is cleared first, so padding bits and bytes are zero. */
void orc_pack(const uint8_t *codes, int64_t n, int bits, uint8_t *out, int64_t out_bytes)
{
    memset(out, 0, (size_t)out_bytes);
    for (int64_t j = 0; j < n; ++j) {
        for (int b = 0; b < bits; ++b) {
            if ((codes[j] >> b) & 1u) {
                int64_t pos = j * bits + b;
                out[pos >> 3] |= (uint8_t)(1u << (pos & 7));
            }
        }
    }
}

void orc_unpack(const uint8_t *packed, int64_t n, int bits, uint8_t *codes)
{
    for (int64_t j = 0; j < n; ++j) {
        unsigned c = 0;
        for (int b = 0; b < bits; ++b) {
            int64_t pos = j * bits + b;
            c |= (unsigned)((packed[pos >> 3] >> (pos & 7)) & 1u) << b;
        }
        codes[j] = (uint8_t)c;
    }
}

/* Matrix operand: rows x cols codes, each row its own bit stream starting
 * at a multiple of row_stride bytes; the tail of every row is zero bits
 * (code 0, value 0). */
void orc_pack_rows(const uint8_t *codes, int64_t rows, int64_t cols, int bits,
                   uint8_t *out, int64_t row_stride)
{
    for (int64_t r = 0; r < rows; ++r)
        orc_pack(codes + r * cols, cols, bits, out + r * row_stride, row_stride);
}

void orc_unpack_rows(const uint8_t *packed, int64_t rows, int64_t cols, int bits,
                     int64_t row_stride, uint8_t *codes)
{
    for (int64_t r = 0; r < rows; ++r)
        orc_unpack(packed + r * row_stride, cols, bits, codes + r * cols);
}

/* ------------------------------------------------------------------ */
/* Dequantise                                                          */
/* ------------------------------------------------------------------ */

/* out[i] = scale * value(code[i]), one fp32 multiply (the value is exact
 * in fp32). */
void orc_dequantize(const uint8_t *codes, int64_t n, int bits, int is_signed,
                    float scale, float *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = scale * (float)orc_decode(bits, is_signed, codes[i]);
}

/* ------------------------------------------------------------------ */
/* GEMM on coded operands (Section III-B.1: the array computes the      */
/* layer's sum of products on decoded values)                          */
/* ------------------------------------------------------------------ */

/* Integer image of a code: value * 2^(m-1), exact (every DyBit value is a
 * multiple of 2^-(m-1)). */
static int64_t code_int(int bits, int is_signed, unsigned code)
{
    int m = mag_bits(bits, is_signed);
    return (int64_t)llround(ldexp(orc_decode(bits, is_signed, code), m - 1));
}

/* All 2^bits integer images of a format, enumerated once per call. */
static void int_table(int bits, int is_signed, int64_t *tab /* 256 */)
{
    for (unsigned c = 0; c < 256u; ++c)
        tab[c] = (c < (1u << bits)) ? code_int(bits, is_signed, c) : 0;
}

/* alpha folds both scales and both integer rescales into one fp32 factor. */
float orc_alpha(float scale_a, int bits_a, int signed_a,
                float scale_b, int bits_b, int signed_b)
{
    int ea = mag_bits(bits_a, signed_a) - 1, eb = mag_bits(bits_b, signed_b) - 1;
    return (float)ldexp((double)scale_a * (double)scale_b, -(ea + eb));
}

/* A: M x K codes, B: N x K codes (both K-contiguous, i.e. C = A * B^T).
 * S[i][j] = sum_k IA[i][k] * IB[j][k] exactly in int64 (optional output);
 * C[i][j] = (float)S * alpha: one int->float conversion (round to nearest
 * even) and one fp32 multiply. */
void orc_gemm(int64_t M, int64_t N, int64_t K,
              const uint8_t *A, int bits_a, int signed_a, float scale_a,
              const uint8_t *B, int bits_b, int signed_b, float scale_b,
              int64_t *S, float *C)
{
    float alpha = orc_alpha(scale_a, bits_a, signed_a, scale_b, bits_b, signed_b);
    int64_t ta[256], tb[256];
    int_table(bits_a, signed_a, ta);
    int_table(bits_b, signed_b, tb);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            int64_t acc = 0;
            for (int64_t k = 0; k < K; ++k)
                acc += ta[A[i * K + k]] * tb[B[j * K + k]];
            if (S) S[i * N + j] = acc;
            if (C) C[i * N + j] = (float)acc * alpha;
        }
    }
}

/* Same definition for chosen output entries only: entry e is
 * (rows_idx[e], cols_idx[e]).  Lets a test check sampled outputs of a
 * GEMM that is too large to recompute in full. */
void orc_gemm_sampled(int64_t N, int64_t K,
                      const uint8_t *A, int bits_a, int signed_a, float scale_a,
                      const uint8_t *B, int bits_b, int signed_b, float scale_b,
                      const int64_t *rows_idx, const int64_t *cols_idx, int64_t n_samples,
                      int64_t *S, float *C)
{
    (void)N;
    float alpha = orc_alpha(scale_a, bits_a, signed_a, scale_b, bits_b, signed_b);
    int64_t ta[256], tb[256];
    int_table(bits_a, signed_a, ta);
    int_table(bits_b, signed_b, tb);
#pragma omp parallel for schedule(static)
    for (int64_t e = 0; e < n_samples; ++e) {
        int64_t i = rows_idx[e], j = cols_idx[e];
        int64_t acc = 0;
        for (int64_t k = 0; k < K; ++k)
            acc += ta[A[i * K + k]] * tb[B[j * K + k]];
        if (S) S[e] = acc;
        if (C) C[e] = (float)acc * alpha;
    }
}

/* ------------------------------------------------------------------ */
/* Convolution on coded operands, the direct definition                */
/* (Section III-C.4 maps layers onto the GEMM array; the result is the  */
/* layer's own sum over taps and channels)                             */
/* ------------------------------------------------------------------ */

/* X: [n][h][w][c] codes; W: [k][r][s][c] codes; Y: [n][oh][ow][k].
 * Taps outside the image contribute 0. */
void orc_conv2d(int n, int h, int w, int c, int k, int r, int s,
                int stride, int pad, int dilation,
                const uint8_t *X, int bits_x, int signed_x, float scale_x,
                const uint8_t *W, int bits_w, int signed_w, float scale_w,
                int64_t *S, float *Y)
{
    int oh = (h + 2 * pad - dilation * (r - 1) - 1) / stride + 1;
    int ow = (w + 2 * pad - dilation * (s - 1) - 1) / stride + 1;
    float alpha = orc_alpha(scale_x, bits_x, signed_x, scale_w, bits_w, signed_w);
    int64_t tx[256], tw[256];
    int_table(bits_x, signed_x, tx);
    int_table(bits_w, signed_w, tw);
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in) {
        for (int io = 0; io < oh; ++io) {
            for (int jo = 0; jo < ow; ++jo) {
                for (int ko = 0; ko < k; ++ko) {
                    int64_t acc = 0;
                    for (int ir = 0; ir < r; ++ir) {
                        int ih = io * stride - pad + ir * dilation;
                        if (ih < 0 || ih >= h) continue;
                        for (int is = 0; is < s; ++is) {
                            int iw = jo * stride - pad + is * dilation;
                            if (iw < 0 || iw >= w) continue;
                            for (int ic = 0; ic < c; ++ic) {
                                unsigned cx = X[(((int64_t)in * h + ih) * w + iw) * c + ic];
                                unsigned cw = W[(((int64_t)ko * r + ir) * s + is) * c + ic];
                                acc += tx[cx] * tw[cw];
                            }
                        }
                    }
                    int64_t o = (((int64_t)in * oh + io) * ow + jo) * k + ko;
                    if (S) S[o] = acc;
                    if (Y) Y[o] = (float)acc * alpha;
                }
            }
        }
    }
}

/* The same convolution for chosen outputs only, starting from the fp32
 * activation: each needed element is encoded on the spot with
 * orc_encode_one (t = |x| * inv_x), so a test can check sampled outputs of a
 * layer too large to quantise and convolve in full.  idx[e] is the flat index
 * into Y[n][oh][ow][k]. */
void orc_conv2d_sampled(int n, int h, int w, int c, int k, int r, int s,
                        int stride, int pad, int dilation,
                        const float *X, int bits_x, int signed_x, float scale_x, float inv_x,
                        const uint8_t *W, int bits_w, int signed_w, float scale_w,
                        const int64_t *idx, int64_t n_samples, int64_t *S, float *Y)
{
    int oh = (h + 2 * pad - dilation * (r - 1) - 1) / stride + 1;
    int ow = (w + 2 * pad - dilation * (s - 1) - 1) / stride + 1;
    (void)n;
    float alpha = orc_alpha(scale_x, bits_x, signed_x, scale_w, bits_w, signed_w);
    int64_t tx[256], tw[256];
    int_table(bits_x, signed_x, tx);
    int_table(bits_w, signed_w, tw);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t e = 0; e < n_samples; ++e) {
        int64_t o = idx[e];
        int ko = (int)(o % k); o /= k;
        int jo = (int)(o % ow); o /= ow;
        int io = (int)(o % oh); o /= oh;
        int in = (int)o;
        int64_t acc = 0;
        for (int ir = 0; ir < r; ++ir) {
            int ih = io * stride - pad + ir * dilation;
            if (ih < 0 || ih >= h) continue;
            for (int is = 0; is < s; ++is) {
                int iw = jo * stride - pad + is * dilation;
                if (iw < 0 || iw >= w) continue;
                for (int ic = 0; ic < c; ++ic) {
                    float xv = X[(((int64_t)in * h + ih) * w + iw) * c + ic];
                    unsigned cx = orc_encode_one(xv, inv_x, bits_x, signed_x);
                    unsigned cw = W[(((int64_t)ko * r + ir) * s + is) * c + ic];
                    acc += tx[cx] * tw[cw];
                }
            }
        }
        if (S) S[e] = acc;
        if (Y) Y[e] = (float)acc * alpha;
    }
}

/* Depth-wise convolution (the 3x3 layers of MobileNetV2, one of the models of
 * Section IV-A): every channel is filtered by its own r x s kernel, no sum
 * across channels.  X: [n][h][w][c] codes; W: [c][r][s] codes; Y: [n][oh][ow][c].
 * S is the exact integer sum over the taps, Y = (float)S * alpha as in the
 * dense layers. */
void orc_depthwise_conv2d(int n, int h, int w, int c, int r, int s,
                          int stride, int pad, int dilation,
                          const uint8_t *X, int bits_x, int signed_x, float scale_x,
                          const uint8_t *W, int bits_w, int signed_w, float scale_w,
                          int64_t *S, float *Y)
{
    int oh = (h + 2 * pad - dilation * (r - 1) - 1) / stride + 1;
    int ow = (w + 2 * pad - dilation * (s - 1) - 1) / stride + 1;
    float alpha = orc_alpha(scale_x, bits_x, signed_x, scale_w, bits_w, signed_w);
    int64_t tx[256], tw[256];
    int_table(bits_x, signed_x, tx);
    int_table(bits_w, signed_w, tw);
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in) {
        for (int io = 0; io < oh; ++io) {
            for (int jo = 0; jo < ow; ++jo) {
                for (int ic = 0; ic < c; ++ic) {
                    int64_t acc = 0;
                    for (int ir = 0; ir < r; ++ir) {
                        int ih = io * stride - pad + ir * dilation;
                        if (ih < 0 || ih >= h) continue;
                        for (int is = 0; is < s; ++is) {
                            int iw = jo * stride - pad + is * dilation;
                            if (iw < 0 || iw >= w) continue;
                            unsigned cx = X[(((int64_t)in * h + ih) * w + iw) * c + ic];
                            unsigned cw = W[((int64_t)ic * r + ir) * s + is];
                            acc += tx[cx] * tw[cw];
                        }
                    }
                    int64_t o = (((int64_t)in * oh + io) * ow + jo) * c + ic;
                    if (S) S[o] = acc;
                    if (Y) Y[o] = (float)acc * alpha;
                }
            }
        }
    }
}

/* ------------------------------------------------------------------ */
/* Quantization error metric, Eq. 2 (Section III-C.1)                  */
/* ------------------------------------------------------------------ */

/* RMSE = sqrt( (1/n) * sum_i ((x_i - xhat_i) / sigma)^2 ), where xhat is the
 * quantize-dequantize image of x under the given format and {scale, inv}
 * and sigma is the standard deviation of the tensor x (population form,
 * mean of squared deviations from the mean).  Everything in double from
 * the fp32 inputs; xhat_i itself is the fp32 value orc_dequantize returns.
 * out[0] = RMSE, out[1] = sigma, out[2] = mean squared error (before the
 * division by sigma^2).  n == 0 or sigma == 0 give RMSE = 0. */
void orc_rmse(const float *x, int64_t n, int bits, int is_signed, float scale, float inv, double *out)
{
    double mean = 0.0, var = 0.0, se = 0.0;
    for (int64_t i = 0; i < n; ++i) mean += (double)x[i];
    if (n > 0) mean /= (double)n;
    for (int64_t i = 0; i < n; ++i) {
        double d = (double)x[i] - mean;
        var += d * d;
        unsigned c = orc_encode_one(x[i], inv, bits, is_signed);
        float xhat = scale * (float)orc_decode(bits, is_signed, c);
        double e = (double)x[i] - (double)xhat;
        se += e * e;
    }
    double sigma = n > 0 ? sqrt(var / (double)n) : 0.0;
    double mse = n > 0 ? se / (double)n : 0.0;
    out[0] = (sigma > 0.0) ? sqrt(mse) / sigma : 0.0;
    out[1] = sigma;
    out[2] = mse;
}

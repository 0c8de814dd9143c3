/*
 * dybit.h -- C ABI of the DyBit quantize/pack + coded-operand GEMM library
 * for NVIDIA B200 (sm_100a).
 *
 * DyBit ("DyBit: Dynamic Bit-Precision Numbers for Efficient Quantized
 * Neural Network Inference", arXiv 2302.12510) is an N-bit number format
 * with an optional sign bit, a unary (leading-ones) exponent field of
 * variable length and the remaining bits as fraction (Section III-A, Eq. 1,
 * Table I).  A tensor is stored as one per-tensor fp32 scale plus one code
 * per element; real value = scale * value(code).
 *
 * Conventions for every entry point
 *   - Pointers marked [dev] are device pointers, [host] host pointers.  The
 *     caller owns every buffer, including workspace; the library allocates
 *     no device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Device work is enqueued on it and the call returns without waiting.
 *   - Scales live in device memory as two floats: scale[0] = scale,
 *     scale[1] = 1/scale as the encoder uses it.  No host sync is needed
 *     between quantize and GEMM.
 *   - Every function returns a dybit_status; argument errors are detected
 *     before anything is launched.  Nothing aborts or throws.
 *   - A code width `bits` is 2..8.  Signed formats spend the top bit on the
 *     sign and have m = bits-1 magnitude bits; unsigned formats have
 *     m = bits.  "Code 0" is the all-zero pattern and decodes to exactly 0.
 */
#ifndef DYBIT_H_
#define DYBIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DYBIT_OK = 0,
    DYBIT_ERR_INVALID_ARG = 1,    /* null pointer, negative size, bits outside 2..8 ...      */
    DYBIT_ERR_UNSUPPORTED = 2,    /* valid but not implemented (e.g. K beyond int32 headroom) */
    DYBIT_ERR_ALIGNMENT = 3,      /* a pointer or stride is not aligned as documented         */
    DYBIT_ERR_WORKSPACE = 4,      /* workspace missing or smaller than the *_workspace_bytes  */
    DYBIT_ERR_CUDA = 5,           /* a CUDA runtime / driver call failed                      */
    DYBIT_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait expired (see dybit_last_device_status) */
    DYBIT_ERR_DEVICE_BOUNDS = 7   /* debug build only (libdybit_debug.so): a range check skipped an access       */
} dybit_status;

/* One tensor's code format (Section III-A). */
typedef struct {
    int bits;       /* total code width, 2..8                                   */
    int is_signed;  /* 1: MSB is the sign, bits-1 magnitude bits; 0: all magnitude */
} dybit_fmt;

/* Tensor-core input type the GEMM expands codes into: the narrowest type
 * that holds every value of both operand formats exactly (Section III-B.3
 * picks a multiplier mode per bitwidth pair; this is its analogue). */
typedef enum {
    DYBIT_CONTAINER_I8 = 0,    /* int8 x int8 -> int32, exact                */
    DYBIT_CONTAINER_E4M3 = 1,  /* fp8 e4m3 x e4m3 -> fp32                    */
    DYBIT_CONTAINER_BF16 = 2   /* bf16 x bf16 -> fp32                        */
} dybit_container;

/* Convolution geometry: X is [n][h][w][c] (NHWC), W is [k][r][s][c],
 * Y is [n][oh][ow][k] with oh = (h + 2*pad - dilation*(r-1) - 1)/stride + 1
 * (ow likewise).  Taps outside the image contribute 0. */
typedef struct {
    int n, h, w, c;
    int k, r, s;
    int stride, pad, dilation;
} dybit_conv_desc;

/* ---------------------------------------------------------------- host-only helpers */

/* Static, NUL-terminated description of a status code. */
const char *dybit_status_string(dybit_status st);

/* Bytes of a packed 1-D tensor of n codes: ceil(n*bits/8) rounded up to 16.
 * Returns 0 for invalid arguments. */
size_t dybit_packed_bytes(int64_t n, int bits);

/* Row stride, in bytes, of a packed matrix operand with k columns: k is
 * padded up to a multiple of 128 codes, so the stride is a multiple of
 * 16 bytes.  Returns 0 for invalid arguments. */
size_t dybit_row_stride_bytes(int64_t k, int bits);

/* Eq. 1 enumerated: table[c] = value of code c for c < 2^bits, 0 above.
 * table: [host] 256 floats. */
dybit_status dybit_decode_table(dybit_fmt fmt, float *table);

/* Enumerates both formats' value tables and reports the container the GEMM
 * will use for this pair, plus the power-of-two exponents by which each
 * operand's values are multiplied before conversion (int8 container only:
 * value * 2^exp is an integer; 0 for the floating containers).
 * All three outputs: [host], each may be NULL. */
dybit_status dybit_choose_container(dybit_fmt fa, dybit_fmt fb, dybit_container *container,
                                    int *exp_a, int *exp_b);

/* Workspace sizes (bytes) the caller must provide to dybit_gemm /
 * dybit_conv2d.  0 is returned for invalid arguments; a valid problem never
 * needs 0 bytes. */
size_t dybit_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, dybit_fmt fa, dybit_fmt fb);
size_t dybit_conv2d_workspace_bytes(const dybit_conv_desc *desc, dybit_fmt fx, dybit_fmt fw);

/* Output spatial size of a convolution.  oh / ow: [host]. */
dybit_status dybit_conv2d_out_hw(const dybit_conv_desc *desc, int *oh, int *ow);

/* ---------------------------------------------------------------- device entry points */

/* Per-tensor max-abs scale (Section I: the format adjusts its precision at
 * the tensor level).  amax = largest finite |x|;
 * scale_out[0] = amax / 2^(m-1), scale_out[1] = 2^(m-1) / amax (one fp32
 * division).  amax == 0 (or n == 0) gives {1, 1}.
 *   x         [dev]  n floats, 4-byte aligned (16-byte aligned runs fastest)
 *   scale_out [dev]  2 floats, overwritten                                  */
dybit_status dybit_absmax_scale(const float *x, int64_t n, dybit_fmt fmt, float *scale_out,
                                void *stream);

/* Quantize + pack a 1-D tensor (Section III-A format; encoder of
 * Section III-B.2).  Per element: t = |x| * scale[1] in fp32; magnitude code
 * = the code whose value is nearest to t (ties to the even code; t beyond
 * the largest value saturates to all-ones; NaN -> code 0); the sign bit is
 * the sign of x unless the magnitude code is 0; an unsigned format maps
 * negative x to code 0.  Codes are written as a dense little-endian bit
 * stream: code j occupies stream bits [j*bits, (j+1)*bits), stream bit b is
 * bit b%8 of byte b/8.  Bits past the last code, up to
 * dybit_packed_bytes(n, bits), are written as zero.
 *   x         [dev]  n floats, 4-byte aligned
 *   scale     [dev]  2 floats {scale, 1/scale}, or NULL: the max-abs scale
 *                    is computed first and written to scale_out (which must
 *                    then be non-NULL)
 *   packed    [dev]  dybit_packed_bytes(n, bits) bytes, 16-byte aligned
 *   scale_out [dev]  2 floats or NULL; receives the scale that was used     */
dybit_status dybit_quantize_pack(const float *x, int64_t n, dybit_fmt fmt, const float *scale,
                                 void *packed, float *scale_out, void *stream);

/* Quantize + pack a matrix operand for dybit_gemm: rows x cols fp32, row r
 * starting at x + r*ld, into rows of row_stride_bytes each; every row is
 * its own bit stream and is zero-filled (code 0) from column `cols` to the
 * end of the row.  With scale == NULL one max-abs scale over the whole
 * matrix is computed first.
 *   ld               in floats, >= cols
 *   row_stride_bytes multiple of 16, >= dybit_row_stride_bytes(cols, bits) */
dybit_status dybit_quantize_pack_2d(const float *x, int64_t rows, int64_t cols, int64_t ld,
                                    dybit_fmt fmt, const float *scale, void *packed,
                                    int64_t row_stride_bytes, float *scale_out, void *stream);

/* Decode a packed 1-D tensor (decoder of Section III-B.2, as the
 * enumerated table of Eq. 1): out[j] = scale[0] * value(code j), one fp32
 * multiply.
 *   packed [dev] dybit_packed_bytes(n, bits) bytes, 16-byte aligned
 *   scale  [dev] 2 floats (only scale[0] is read), or NULL for scale 1
 *   out    [dev] n floats                                                   */
dybit_status dybit_decode(const void *packed, int64_t n, dybit_fmt fmt, const float *scale,
                          float *out, void *stream);

/* Matrix multiply on coded operands (the array of Section III-B.1 computes
 * a layer as the sum of products of decoded values; Section III-B.3 picks
 * the multiplier mode from the two bitwidths):
 *     C[i][j] = sA * sB * sum_k value_A(A[i][k]) * value_B(B[j][k])
 * Both operands are K-contiguous packed matrices (C = A * B^T), as written
 * by dybit_quantize_pack_2d.
 *   A        [dev] M rows of lda_bytes, B [dev] N rows of ldb_bytes; strides
 *            multiples of 16 >= dybit_row_stride_bytes(K, bits); the row
 *            tails past K must hold code 0
 *   scale_a/b [dev] 2 floats each (only [0] is read)
 *   C        [dev] M x N floats, row stride ldc floats (ldc >= N)
 *   C_raw    [dev] optional (may be NULL) M x N int32, row stride ldc: the
 *            exact integer sum of value*2^(m-1) products; only available
 *            with the int8 container (DYBIT_ERR_UNSUPPORTED otherwise)
 *   ws       [dev] dybit_gemm_workspace_bytes(...) bytes, 1024-byte aligned
 * int8 container: C = (float)sum * alpha with
 * alpha = (float)((double)sA*sB*2^-(expA+expB)), bit-exact.  Floating
 * containers accumulate in fp32.  K above 2^19 is rejected for int8. */
dybit_status dybit_gemm(int64_t M, int64_t N, int64_t K,
                        const void *A, dybit_fmt fa, const float *scale_a, int64_t lda_bytes,
                        const void *B, dybit_fmt fb, const float *scale_b, int64_t ldb_bytes,
                        float *C, int64_t ldc, int32_t *C_raw,
                        void *ws, size_t ws_bytes, void *stream);

/* Batched GEMM: `batch` independent products of equal shape, C_b = alpha * A_b * B_b^T for b = 0..batch-1 (the
 * attention products of ViT-Base, one of the models of Section IV-A, are of this kind: 12 heads x batch matrices of
 * 197 x 64).  Each operand is ONE quantized tensor with one scale; entry b of A starts stride_a_bytes after entry
 * b-1 (likewise B; C and C_raw: stride_c elements).  Every entry is tiled on its own, so no tile mixes two entries.
 * Arguments, alignment and exactness as dybit_gemm; additionally stride_a_bytes, stride_b_bytes multiples of 16,
 * stride_a_bytes >= M*lda_bytes, stride_b_bytes >= N*ldb_bytes, stride_c >= (M-1)*ldc + N.  Dense batches
 * (stride == rows * ld) expand in one launch, others entry by entry.
 *   ws [dev] dybit_gemm_batched_workspace_bytes(...) bytes, 1024-byte aligned */
size_t dybit_gemm_batched_workspace_bytes(int64_t batch, int64_t M, int64_t N, int64_t K, dybit_fmt fa, dybit_fmt fb);
dybit_status dybit_gemm_batched(int64_t batch, int64_t M, int64_t N, int64_t K,
                                const void *A, dybit_fmt fa, const float *scale_a, int64_t lda_bytes, int64_t stride_a_bytes,
                                const void *B, dybit_fmt fb, const float *scale_b, int64_t ldb_bytes, int64_t stride_b_bytes,
                                float *C, int64_t ldc, int64_t stride_c, int32_t *C_raw,
                                void *ws, size_t ws_bytes, void *stream);

/* Convolution on coded operands as an implicit GEMM (Section III-C.4: conv
 * and FC layers run on the GEMM dataflow), M = n*oh*ow, N = k, K = r*s*c:
 *     Y[n][oh][ow][k] = sX*sW * sum_{r,s,c} value(X[n][ih][iw][c]) * value(W[k][r][s][c])
 *   X     [dev] NHWC codes as ONE dense 1-D stream of n*h*w*c codes
 *         (dybit_quantize_pack of the NHWC tensor), 16-byte aligned
 *   W     [dev] k rows of r*s*c codes, row stride ldw_bytes
 *         (dybit_quantize_pack_2d with rows = k, cols = r*s*c)
 *   Y     [dev] n*oh*ow*k floats, dense;  Y_raw as C_raw above
 *   ws    [dev] dybit_conv2d_workspace_bytes(...) bytes, 1024-byte aligned  */
dybit_status dybit_conv2d(const dybit_conv_desc *desc,
                          const void *X, dybit_fmt fx, const float *scale_x,
                          const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes,
                          float *Y, int32_t *Y_raw,
                          void *ws, size_t ws_bytes, void *stream);

/* The two halves of the path in one call: quantize + pack an fp32 NHWC activation (Section III-A) and run the
 * convolution on its codes (Section III-C.4).  Results are those of dybit_quantize_pack(X) followed by dybit_conv2d,
 * bit for bit: X_packed receives the dense code stream, scale_x_out the pair it was made with, Y the layer's output.
 * What is saved is launches: where the expanded activation is the code order itself (channels a multiple of 16, no
 * patch matrix), one kernel writes the codes, their tensor-core elements and the expanded weights.
 *   X           [dev] n*h*w*c floats, NHWC, 4-byte aligned
 *   scale_x     [dev] {scale, 1/scale} to use, or NULL for the max-abs scale of X
 *   scale_x_out [dev] 2 floats, required (may be scale_x itself)
 *   X_packed    [dev] dybit_packed_bytes(n*h*w*c, fx.bits) bytes, 16-byte aligned, required
 * Everything else as in dybit_conv2d (same workspace size). */
dybit_status dybit_quantize_conv2d(const dybit_conv_desc *desc,
                                   const float *X, dybit_fmt fx, const float *scale_x, float *scale_x_out, void *X_packed,
                                   const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes,
                                   float *Y, int32_t *Y_raw, void *ws, size_t ws_bytes, void *stream);

/* dybit_quantize_conv2d for SEVERAL layers whose inputs do not depend on one another (the branches of a block, the
 * layers of a benchmark that feeds every layer its own activation; Section III-D treats the layers of a model one by
 * one in the same way): the work in front of the tensor cores is folded into few launches, since for the short
 * tensors of the later layers a launch costs more than the data.  One struct per layer, fields as the arguments of
 * dybit_quantize_conv2d; every layer needs its OWN workspace, which stays in use from the first call below until its
 * dybit_conv2d_prepared has run.
 *
 * dybit_quantize_expand_layers: ONE max-abs launch for all layers with scale_x == NULL (per 32 layers), then one
 *   quantize + expand launch per group of layers with the same pair of formats: writes every layer's X_packed,
 *   scale_x_out and, in its workspace, the operands of its tensor-core kernel.  Everything on `stream`.
 * dybit_conv2d_prepared: the rest of one layer (its tensor-core kernel, and the patch gather where the lowering has
 *   one), on any stream that is ordered after the call above.
 * Together they give, bit for bit, what dybit_quantize_conv2d (with Q set: dybit_quantize_conv2d_requant) gives for
 * each layer.
 * DYBIT_ERR_UNSUPPORTED (nothing launched) when a layer's lowering is not one whose quantize launch also writes the
 * expanded operands (channels neither a multiple of 16 nor at most 4 with one-byte elements): use
 * dybit_quantize_conv2d for such a layer. */
typedef struct {
    dybit_conv_desc desc;
    const float *X;              /* [dev] n*h*w*c floats */
    dybit_fmt fx;
    const float *scale_x;        /* [dev] pair to use, or NULL for the max-abs scale */
    float *scale_x_out;          /* [dev] 2 floats, required */
    void *X_packed;              /* [dev] dybit_packed_bytes(n*h*w*c, fx.bits) bytes, required */
    const void *W;               /* [dev] packed weights, k rows */
    dybit_fmt fw;
    const float *scale_w;
    int64_t ldw_bytes;
    float *Y;                    /* [dev] n*oh*ow*k floats (unused when Q is set) */
    int32_t *Y_raw;              /* [dev] or NULL (must be NULL when Q is set) */
    void *ws;                    /* [dev] dybit_conv2d_workspace_bytes(...) bytes of this layer's own */
    size_t ws_bytes;
    /* Q != NULL: the layer leaves through the re-quantizing epilogue instead, as in dybit_conv2d_requant */
    void *Q;                     /* [dev] packed output codes, or NULL for the fp32 output Y */
    dybit_fmt fq;
    const float *scale_q;        /* [dev] {scale, 1/scale} of the output tensor */
    const float *bias;           /* [dev] k floats or NULL */
    int relu;
} dybit_conv_layer;

dybit_status dybit_quantize_expand_layers(const dybit_conv_layer *layers, int n_layers, void *stream);
dybit_status dybit_conv2d_prepared(const dybit_conv_layer *layer, void *stream);
/* dybit_conv2d_prepared for all the layers on one stream, with the tensor-core work of layers that run on the same
 * kernel configuration (4-bit-class formats on the int8 path: halo-tile, im2col and row-major lowerings) folded into
 * shared launches of up to 16 layers: every layer gets a share of the SMs in proportion to its work and its CTAs walk
 * its own tiles as they would in a launch of their own, so results are the same bits.  Layers that do not fit this
 * (other element types, gather lowerings) are launched one by one, in order. */
dybit_status dybit_conv2d_prepared_layers(const dybit_conv_layer *layers, int n_layers, void *stream);

/* Depth-wise convolution on coded operands (MobileNetV2, one of the models of Section IV-A, is built from 3x3
 * layers of this kind): channel ch of the output is channel ch of the input filtered by its own r x s kernel,
 *     Y[n][oh][ow][ch] = sX*sW * sum_{r,s} value(X[n][ih][iw][ch]) * value(W[ch][r][s])
 * desc->k must equal desc->c.  There is no contraction over channels, hence no tensor-core work: the kernel decodes
 * the packed codes itself, accumulates in fp32 on integer values (bit-exact whenever both formats have at most 4
 * magnitude bits; wider formats may round once sums exceed 2^24: |err| <= 1e-5 * r*s * max|x| * max|w|) and is
 * bound by the fp32 output stream.  No workspace.
 *   X   [dev] dense NHWC code stream as for dybit_conv2d, 4-byte aligned
 *   W   [dev] c rows of r*s codes (tap order r, s), row stride ldw_bytes >= dybit_packed_bytes(r*s, fw.bits)
 *   Y   [dev] n*oh*ow*c floats, dense
 * Filters or strides whose staged input patch exceeds 200 KB of shared memory -> DYBIT_ERR_UNSUPPORTED. */
dybit_status dybit_depthwise_conv2d(const dybit_conv_desc *desc,
                                    const void *X, dybit_fmt fx, const float *scale_x,
                                    const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes,
                                    float *Y, void *stream);

/* Quantization error metric of Eq. 2 (Section III-C.1), the quantity the bitwidth search ranks layers by:
 *     RMSE = sqrt( (1/n) * sum_i ((x_i - xhat_i) / sigma)^2 )
 * with xhat_i = scale[0] * value(encode(x_i)) the quantize-dequantize image under `fmt` and {scale, 1/scale}, and
 * sigma the standard deviation of x (population form).  One pass over x; sums are kept in fp64.
 *   x     [dev] n floats;  scale [dev] 2 floats {scale, 1/scale}
 *   out   [dev] 4 doubles, 8-byte aligned: {RMSE, sigma, mean squared error, n}; RMSE = 0 when sigma == 0 or n == 0 */
dybit_status dybit_rmse(const float *x, int64_t n, dybit_fmt fmt, const float *scale, double *out, void *stream);

/* Eq. 2 for up to DYBIT_RMSE_MAX_CANDIDATES candidate (format, scale) pairs in ONE pass over x: the sweep behind
 * the choice of a tensor's bitwidth (the RMSE_i table of Algorithm 1) and of its scale (the tensor-level precision
 * adjustment of Section III-A).  x is read once; every candidate's error is the one dybit_rmse would report.
 *   fmts   [host] n_cand formats
 *   scales [dev]  n_cand pairs {scale, 1/scale}, 2 * n_cand floats
 *   out    [dev]  4 * n_cand doubles, 8-byte aligned: {RMSE, sigma, mse, n} per candidate
 *   best   [dev]  optional (may be NULL): index of the candidate with the smallest RMSE, lowest index among equals
 * n == 0 gives all zeros and best = 0.  n_cand outside 1..DYBIT_RMSE_MAX_CANDIDATES -> DYBIT_ERR_INVALID_ARG. */
#define DYBIT_RMSE_MAX_CANDIDATES 16
dybit_status dybit_rmse_sweep(const float *x, int64_t n, int n_cand, const dybit_fmt *fmts, const float *scales,
                              double *out, int *best, void *stream);

/* Fake quantization, the forward of quantization-aware training (Section IV-A fine-tunes the quantized models for
 * a few epochs; the paper does not spell the operator out, this is the usual one): the fp32 image of x under the
 * format, y_i = fmul_rn(scale[0], value(encode(x_i, scale[1]))), i.e. dybit_decode(dybit_quantize_pack(x)) in one
 * streaming pass that never stores the codes.  NaN -> 0, as in the encoder.
 *   x, y [dev] n floats (y may be x);  scale [dev] {scale, 1/scale} */
dybit_status dybit_fake_quant(const float *x, int64_t n, dybit_fmt fmt, const float *scale, float *y, void *stream);

/* Backward of dybit_fake_quant by the straight-through estimator with clipping (a reading: the paper trains with
 * QAT but gives no gradient rule): gx_i = gy_i where lo <= x_i <= hi, else 0, with hi = fmul_rn(scale[0], 2^(m-1))
 * the largest representable value (m magnitude bits) and lo = -hi for a signed format, 0 for an unsigned one.
 * NaN in x gives 0.   x, gy, gx [dev] n floats (gx may be gy) */
dybit_status dybit_fake_quant_backward(const float *x, const float *gy, int64_t n, dybit_fmt fmt, const float *scale,
                                       float *gx, void *stream);

/* Layer-wise bitwidth search of Algorithm 1 (Section III-C.3) -- host only.  All layers start at (8, 8); each
 * round ranks the layers that can still be degraded (speedup strategy: the top_k slowest, re-ordered by ascending
 * RMSE; RMSE strategy: the top_k with the smallest RMSE, re-ordered by descending latency) and degrades first the
 * weights, then the activations of that list one layer at a time (8 -> 4 -> 2), re-evaluating the total after every
 * single step, until the constraint is met:
 *   strategy 0 (speedup, Eq. 3): stop when constraint * sum Lat_i(a, w) <= sum Lat_i(8, 8)        (constraint = alpha)
 *   strategy 1 (RMSE,    Eq. 4): keep degrading while sum RMSE_i(a, w) <= constraint * sum RMSE_i(8, 8); the step
 *                                that would exceed the budget is taken back                      (constraint = beta)
 * or until every layer is at (2, 2).
 *   lat, rmse  [host] num_layers * 9 doubles, index (layer * 3 + a_idx) * 3 + w_idx with idx 0, 1, 2 <-> 8, 4, 2 bits
 *              (latencies e.g. measured per layer with dybit_conv2d, errors with dybit_rmse)
 *   w_bits, a_bits [host] num_layers ints each, receive 8, 4 or 2 */
dybit_status dybit_search_bitwidths(int num_layers, const double *lat, const double *rmse, int strategy,
                                    double constraint, int top_k, int *w_bits, int *a_bits);

/* GEMM / convolution with the re-quantizing epilogue of Section III-B.1 (the accelerator encodes its floating-point
 * intermediate results as DyBit before it writes them to memory): instead of fp32, the result leaves the kernel as
 * packed DyBit codes of format fq, ready to be the next layer's activation.  Per output element (row m, column j)
 *     y = fmul_rn((float)sum, alpha)            exactly as dybit_gemm / dybit_conv2d compute it
 *     y = fadd_rn(y, bias[j])                   if bias != NULL (one fp32 per output column / channel, e.g. a
 *                                               folded batch-norm shift)
 *     y = max(y, 0)                             if relu != 0
 *     code = encode(y, scale_q[1])              the encoder of dybit_quantize_pack (nearest value, ties to even code)
 * and row m of the output (N codes; N = desc->k for the convolution) is written as a dense little-endian bit
 * stream starting at Q + m * ldq_bytes.
 *   scale_q [dev] {scale, 1/scale} of the OUTPUT tensor, given by the caller (e.g. a calibrated or trained scale;
 *           the maximum of the result is not known before it is computed)
 *   bias    [dev] N floats, 4-byte aligned, or NULL
 *   Q       [dev] M rows of ldq_bytes; ldq_bytes >= N*fq.bits/8 and N*fq.bits a multiple of 8 (rows that start on
 *           4-byte boundaries are written with word stores, others byte by byte).  Only the first N*fq.bits/8 bytes of each row are written: a caller that wants padded
 *           rows (ldq_bytes = dybit_row_stride_bytes(N, fq.bits), to feed dybit_gemm) zero-fills the buffer once.
 *           dybit_conv2d_requant writes the dense NHWK stream (ldq_bytes = k*fq.bits/8), which is exactly the X
 *           argument of the next dybit_conv2d.
 * Everything else as in dybit_gemm / dybit_conv2d (same workspace sizes).  int8-container results are bit-exact. */
dybit_status dybit_gemm_requant(int64_t M, int64_t N, int64_t K,
                                const void *A, dybit_fmt fa, const float *scale_a, int64_t lda_bytes,
                                const void *B, dybit_fmt fb, const float *scale_b, int64_t ldb_bytes,
                                dybit_fmt fq, const float *scale_q, const float *bias, int relu, void *Q,
                                int64_t ldq_bytes,
                                void *ws, size_t ws_bytes, void *stream);
dybit_status dybit_conv2d_requant(const dybit_conv_desc *desc,
                                  const void *X, dybit_fmt fx, const float *scale_x,
                                  const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes,
                                  dybit_fmt fq, const float *scale_q, const float *bias, int relu, void *Q,
                                  void *ws, size_t ws_bytes, void *stream);

/* One whole layer of Section III-B.1 in one call: the fp32 NHWC activation is quantized and packed
 * (dybit_quantize_conv2d's arguments X, scale_x, scale_x_out, X_packed), convolved on its codes, and the result leaves
 * as packed DyBit codes (dybit_conv2d_requant's arguments fq, scale_q, bias, relu, Q).  Bit for bit the results of
 * dybit_quantize_pack followed by dybit_conv2d_requant; same workspace size as dybit_conv2d. */
dybit_status dybit_quantize_conv2d_requant(const dybit_conv_desc *desc,
                                           const float *X, dybit_fmt fx, const float *scale_x, float *scale_x_out,
                                           void *X_packed,
                                           const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes,
                                           dybit_fmt fq, const float *scale_q, const float *bias, int relu, void *Q,
                                           void *ws, size_t ws_bytes, void *stream);

/* (No counterpart in the paper.)  dybit_gemm for callers that cannot call
 * cudaMalloc -- or any allocator built on it -- at the point where they need
 * a GEMM: code running under a fixed memory budget that was handed out at
 * start-up, plug-ins of a host application that owns all device memory, code
 * on a path where an allocation's implicit synchronisation or possible failure
 * is not acceptable.  Same arguments and same result, bit for bit, as
 * dybit_gemm, minus the workspace: the expanded operands go to a scratch array
 * of DYBIT_STATIC_WS_BYTES that is part of this library's device image.  Every
 * GPU on which the process uses the library holds that array from module load
 * until the process exits.
 *   - Problems with dybit_gemm_workspace_bytes(M, N, K, fa, fb) above
 *     DYBIT_STATIC_WS_BYTES are refused with DYBIT_ERR_WORKSPACE and nothing
 *     is launched (e.g. int8-container operands up to (M + N) * roundup(K,128)
 *     of about 16 Mi elements fit).
 *   - The call itself allocates nothing and frees nothing.  The first call on
 *     each device looks up the array's device address (cudaGetSymbolAddress,
 *     with that device current) and remembers it; make that first call outside
 *     any stream capture.
 *   - All calls on a device share the one array.  Nothing in it has to be
 *     zero beforehand and nothing is kept between calls: each call rewrites
 *     every byte it later reads.  Two calls whose device work overlaps (two
 *     streams, or two host threads) would overwrite each other's operands:
 *     keep calls to this entry point ordered on one stream per device. */
#define DYBIT_STATIC_WS_BYTES (16u * 1024u * 1024u)
dybit_status dybit_gemm_static_ws(int64_t M, int64_t N, int64_t K,
                                  const void *A, dybit_fmt fa, const float *scale_a, int64_t lda_bytes,
                                  const void *B, dybit_fmt fb, const float *scale_b, int64_t ldb_bytes,
                                  float *C, int64_t ldc, int32_t *C_raw, void *stream);

/* Reads and clears the device status word of the current device.  Blocks
 * until `stream` has drained.  DYBIT_ERR_DEVICE_TIMEOUT means a kernel gave
 * up on a bounded wait (results of that call are invalid); DYBIT_OK
 * otherwise.  detail: [host] optional, receives the raw status word. */
dybit_status dybit_last_device_status(void *stream, uint32_t *detail);

/* Self-test of the give-up path of the bounded device-side waits (no counterpart in the paper).  Launches one small
 * kernel in which a single thread waits, with the same routine every kernel of the library waits with, on a barrier
 * that nothing will ever signal, for at most limit_ns nanoseconds (1 .. 100,000,000).  The wait runs out, the
 * kernel records it in the device status word and returns normally: afterwards dybit_last_device_status reports
 * DYBIT_ERR_DEVICE_TIMEOUT once (detail = 0x5e01) and the device keeps working.  result: [device] two 32-bit words,
 * [0] = 1 if the wait reported failure, [1] = the CTA's abort flag.  Errors: INVALID_ARG (null result, limit out of
 * range), ALIGNMENT, CUDA. */
dybit_status dybit_selftest_wait_timeout(uint64_t limit_ns, uint32_t *result, void *stream);

/* ---------------------------------------------------------------- measurement hooks
 * (no counterpart in the paper: they exist so that a benchmark can attribute
 * time to the tensor-core kernel alone and count the library's launches) */

/* Process-wide state.  The library keeps none that a result depends on: plans and element tables are cached per
 * format pair and per device (filled on first use, atomically, every thread computing the same values), kernels
 * launched are counted in one atomic counter, and the device status word lives in the loaded module.  The two
 * dybit_profile_next_gemm* hooks below arm state that is PER HOST THREAD (the arming thread's next GEMM / conv call
 * consumes it); dybit_set_conv_lowering and dybit_set_gemm_decode are process-wide atomic settings. */

/* Which lowering dybit_conv2d and its variants take for stride-1 convolutions (Section III-C.4 maps conv layers onto
 * the GEMM array; the lowerings differ only in how the activation tile reaches shared memory, never in results):
 *   0 (default)  choose by shape: halo tiles where they measured faster (64-byte pixels, one tile column of output
 *                channels whose weights stay resident in shared memory), the im2col / gather lowering otherwise;
 *   1            halo tiles wherever they apply (stride 1, dilation 1, at most three filter rows, pixels of 64 or a
 *                multiple of 128 container bytes);
 *   2            never halo tiles.
 * Returns DYBIT_ERR_INVALID_ARG for any other value.  Takes effect for calls that start afterwards. */
dybit_status dybit_set_conv_lowering(int mode);

/* Where dybit_gemm decodes its B operand (the weights) when B is a 4-bit format in the int8 container and the output
 * is plain fp32 (Section III-B.1-2: decoders beside the array feed it directly):
 *   0  both operands are expanded into the workspace by a separate launch, the GEMM kernel reads those copies;
 *   1  B stays packed and is decoded in the GEMM kernel's main loop (table lookup in registers into the shared-memory
 *      operand tile) wherever that kernel applies;
 *   2 (default)  by shape: in the main loop when A has at most 128 rows and B at least 32 Mi codes (the GEMM is then
 *      bound by the one pass over the weights, which shrinks from 2.5 to 0.5 bytes per weight), expanded otherwise.
 * Results are identical bit for bit in every mode.  Returns DYBIT_ERR_INVALID_ARG for any other value. */
dybit_status dybit_set_gemm_decode(int mode);

/* Number of kernels this library has launched in the calling process so far. */
uint64_t dybit_launch_count(void);

/* Arms the calling thread: the next dybit_gemm / dybit_conv2d records
 * ev_start on its stream immediately before its tensor-core kernel and
 * ev_stop immediately after it (the expand kernels stay outside the pair),
 * then disarms.  Both are cudaEvent_t passed as void*; NULL, NULL disarms. */
dybit_status dybit_profile_next_gemm(void *ev_start, void *ev_stop);

/* The same arming for the device's own clock: the CTAs of the next
 * tensor-core kernel min-reduce the time at which they pass the dependency
 * wait into t2[0] and max-reduce the time at which they retire into t2[1]
 * (nanoseconds of %globaltimer; device memory, 8-byte aligned, initialised
 * by the caller to {UINT64_MAX, 0}).  Unlike an event pair this brackets the
 * kernel's own run even inside a CUDA graph replay, where neighbouring
 * launches overlap its prologue; stores still in flight when the last CTA
 * retires are not covered.  NULL disarms. */
dybit_status dybit_profile_next_gemm_clock(unsigned long long *t2);

#ifdef __cplusplus
}
#endif
#endif /* DYBIT_H_ */

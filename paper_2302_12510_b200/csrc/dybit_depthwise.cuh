// Depth-wise convolution on DyBit-coded operands (the 3x3 layers of MobileNetV2, Section IV-A):
// every channel is filtered by its own r x s kernel, so there is no contraction a tensor core could
// carry -- r*s multiply-adds per output against 4 bytes written.  The kernel is bound by the fp32
// output stream; it decodes the packed codes itself, once per staged input element.
//
// One block = one image, one 8 x 8 tile of output pixels, one slab of 32 channels:
//   1. the input patch the tile needs ((8-1)*stride + (r-1)*dilation + 1 rows and columns, zeros
//      outside the image) is decoded from the packed NHWC stream into shared memory as fp32
//      integers value * 2^(m-1), channel innermost;
//   2. the slab's filters are decoded the same way, tap-major;
//   3. warp w owns output row w, lane l channel l: eight outputs per thread, the input row held
//      in registers across the filter columns; one fp32 FMA per tap (exact while the sums stay
//      below 2^24, i.e. always for formats with at most 4 magnitude bits);
//   4. y = fmul_rn(sum, alpha): each warp writes 128 contiguous bytes per output pixel.
#pragma once

#include "dybit_common.cuh"
#include "dybit_host.cuh"

namespace dybit {

constexpr int kDwTile = 8;        // output pixels per tile edge (= warps per block)
constexpr int kDwChannels = 32;   // channels per block (= lanes)
constexpr int kDwThreads = kDwTile * 32;

struct DwParams {
    const uint8_t *X, *W;
    float *Y;
    const float *scale_x, *scale_w;
    double pow2;                  // alpha = (float)(scale_x * scale_w * pow2)
    int64_t ldw;
    int x_bits, w_bits;
    int H, Wd, C, R, S, OH, OW, stride, pad, dil;
    int tiles_h, tiles_w, c_tiles;
    int in_h, in_w;               // extent of the staged input patch
    int x_words;                  // X may be read as whole 32-bit words (power-of-two width, word-aligned pixels)
};

struct DwTables {
    float x[256], w[256];         // integer-valued: value(code) * 2^(m-1)
};

// Code number `index` of a dense little-endian stream of `bits`-wide codes (bits <= 8), byte loads only.
__device__ __forceinline__ unsigned stream_code(const uint8_t *__restrict__ base, int64_t index, int bits) {
    const int64_t bitpos = index * bits;
    const int sh = (int)(bitpos & 7);
    unsigned v = __ldg(base + (bitpos >> 3));
    if (sh + bits > 8) v |= (unsigned)__ldg(base + (bitpos >> 3) + 1) << 8;     // the code straddles two bytes
    return (v >> sh) & ((1u << bits) - 1u);
}

// The eight outputs of one thread: RT x ST filter at stride STRIDE, dilation 1, input rows in registers.
template <int RT, int ST, int STRIDE>
__device__ __forceinline__ void dw_accumulate_fixed(const float *__restrict__ s_in, const float *__restrict__ s_w, int in_w,
                                                    int oy, int lane, float (&acc)[kDwTile]) {
    constexpr int NC = (kDwTile - 1) * STRIDE + ST;
#pragma unroll
    for (int r = 0; r < RT; ++r) {
        const float *row = s_in + (size_t)((oy * STRIDE + r) * in_w) * kDwChannels + lane;
        float v[NC];
#pragma unroll
        for (int j = 0; j < NC; ++j) v[j] = row[j * kDwChannels];
#pragma unroll
        for (int s = 0; s < ST; ++s) {
            const float w = s_w[(r * ST + s) * kDwChannels + lane];
#pragma unroll
            for (int j = 0; j < kDwTile; ++j) acc[j] = fmaf(v[j * STRIDE + s], w, acc[j]);
        }
    }
}

__global__ void __launch_bounds__(kDwThreads)
depthwise_kernel(const __grid_constant__ DwParams p, const __grid_constant__ DwTables tab) {
    extern __shared__ __align__(16) float dw_smem[];
    float *s_in = dw_smem;                                         // [in_h][in_w][32]
    float *s_w = dw_smem + (size_t)p.in_h * p.in_w * kDwChannels;  // [R*S][32]
    __shared__ float s_lut_x[256], s_lut_w[256];
    pdl_enter();
    for (int i = threadIdx.x; i < 256; i += blockDim.x) {
        s_lut_x[i] = tab.x[i];
        s_lut_w[i] = tab.w[i];
    }
    int b = blockIdx.x;
    const int ct = b % p.c_tiles;
    b /= p.c_tiles;
    const int tw = b % p.tiles_w;
    b /= p.tiles_w;
    const int th = b % p.tiles_h;
    const int n = b / p.tiles_h;
    const int c0 = ct * kDwChannels;
    const int ih0 = th * kDwTile * p.stride - p.pad, iw0 = tw * kDwTile * p.stride - p.pad;
    __syncthreads();

    // filters of the slab, tap-major
    for (int i = threadIdx.x; i < p.R * p.S * kDwChannels; i += blockDim.x) {
        const int tap = i / kDwChannels, c = c0 + (i % kDwChannels);
        s_w[i] = c < p.C ? s_lut_w[stream_code(p.W + (int64_t)c * p.ldw, tap, p.w_bits)] : 0.0f;
    }
    // input patch
    const int npix = p.in_h * p.in_w;
    if (p.x_words) {
        // one 32-bit word of codes per thread and step: 32 / bits channels of one pixel
        const int per_word = 32 / p.x_bits;
        const int words = (min(kDwChannels, p.C - c0) * p.x_bits + 31) / 32;       // words of this slab per pixel
        const unsigned mask = (1u << p.x_bits) - 1u;
        for (int i = threadIdx.x; i < npix * words; i += blockDim.x) {
            const int pix = i / words, wd = i - pix * words;
            const int iy = pix / p.in_w, ix = pix - iy * p.in_w;
            const int ih = ih0 + iy, iw = iw0 + ix;
            unsigned word = 0u;                                   // code 0 decodes to 0 in every format
            if ((unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.Wd) {
                const int64_t first = (((int64_t)n * p.H + ih) * p.Wd + iw) * p.C + c0;      // code index of the slab
                word = __ldg(reinterpret_cast<const unsigned *>(p.X + first * p.x_bits / 8) + wd);
            }
            float *dst = s_in + (size_t)pix * kDwChannels + wd * per_word;
            const int live = min(per_word, p.C - c0 - wd * per_word);   // channels of this word that exist
            for (int k = 0; k < per_word; ++k) {
                dst[k] = k < live ? s_lut_x[word & mask] : 0.0f;
                word >>= p.x_bits;
            }
        }
        // channels of the slab past C (last slab only) that no word covered
        const int covered = words * per_word;
        if (covered < kDwChannels) {
            const int rest = kDwChannels - covered;
            for (int i = threadIdx.x; i < npix * rest; i += blockDim.x)
                s_in[(size_t)(i / rest) * kDwChannels + covered + (i % rest)] = 0.0f;
        }
    } else {
        for (int i = threadIdx.x; i < npix * kDwChannels; i += blockDim.x) {
            const int pix = i / kDwChannels, c = c0 + (i % kDwChannels);
            const int iy = pix / p.in_w, ix = pix - iy * p.in_w;
            const int ih = ih0 + iy, iw = iw0 + ix;
            float v = 0.0f;
            if (c < p.C && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.Wd)
                v = s_lut_x[stream_code(p.X, (((int64_t)n * p.H + ih) * p.Wd + iw) * p.C + c, p.x_bits)];
            s_in[i] = v;
        }
    }
    __syncthreads();

    const int lane = threadIdx.x & 31, oy = threadIdx.x >> 5;
    float acc[kDwTile];
#pragma unroll
    for (int j = 0; j < kDwTile; ++j) acc[j] = 0.0f;
    if (p.R == 3 && p.S == 3 && p.dil == 1 && p.stride == 1) {
        dw_accumulate_fixed<3, 3, 1>(s_in, s_w, p.in_w, oy, lane, acc);
    } else if (p.R == 3 && p.S == 3 && p.dil == 1 && p.stride == 2) {
        dw_accumulate_fixed<3, 3, 2>(s_in, s_w, p.in_w, oy, lane, acc);
    } else {
        for (int r = 0; r < p.R; ++r) {
            const float *row = s_in + (size_t)((oy * p.stride + r * p.dil) * p.in_w) * kDwChannels + lane;
            for (int s = 0; s < p.S; ++s) {
                const float w = s_w[(r * p.S + s) * kDwChannels + lane];
#pragma unroll
                for (int j = 0; j < kDwTile; ++j) acc[j] = fmaf(row[(j * p.stride + s * p.dil) * kDwChannels], w, acc[j]);
            }
        }
    }
    const float alpha = (float)((double)__ldg(p.scale_x) * (double)__ldg(p.scale_w) * p.pow2);
    const int oh = th * kDwTile + oy, c = c0 + lane;
    if (oh < p.OH && c < p.C) {
        float *yrow = p.Y + (((int64_t)n * p.OH + oh) * p.OW + (int64_t)tw * kDwTile) * p.C + c;
#pragma unroll
        for (int j = 0; j < kDwTile; ++j)
            if (tw * kDwTile + j < p.OW) __stcs(yrow + (int64_t)j * p.C, __fmul_rn(acc[j], alpha));
    }
}

}  // namespace dybit

extern "C" {

dybit_status dybit_depthwise_conv2d(const dybit_conv_desc *d, const void *X, dybit_fmt fx, const float *scale_x,
                                    const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes, float *Y,
                                    void *stream) {
    using namespace dybit;
    int oh, ow;
    dybit_status st = dybit_conv2d_out_hw(d, &oh, &ow);
    if (st != DYBIT_OK) return st;
    if (d->k != d->c) return DYBIT_ERR_INVALID_ARG;               // one filter per channel
    if (!fmt_ok(fx) || !fmt_ok(fw) || !X || !W || !Y || !scale_x || !scale_w) return DYBIT_ERR_INVALID_ARG;
    if (ldw_bytes < (int64_t)dybit_packed_bytes((int64_t)d->r * d->s, fw.bits)) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(X, 4) || !aligned(Y, 4) || !aligned(scale_x, 4) || !aligned(scale_w, 4)) return DYBIT_ERR_ALIGNMENT;
    DwParams p = {};
    p.X = static_cast<const uint8_t *>(X);
    p.W = static_cast<const uint8_t *>(W);
    p.Y = Y;
    p.scale_x = scale_x;
    p.scale_w = scale_w;
    const int mx = fx.bits - (fx.is_signed ? 1 : 0), mw = fw.bits - (fw.is_signed ? 1 : 0);
    p.pow2 = ldexp(1.0, -((mx - 1) + (mw - 1)));
    p.ldw = ldw_bytes;
    p.x_bits = fx.bits;
    p.w_bits = fw.bits;
    p.H = d->h; p.Wd = d->w; p.C = d->c; p.R = d->r; p.S = d->s;
    p.OH = oh; p.OW = ow; p.stride = d->stride; p.pad = d->pad; p.dil = d->dilation;
    p.tiles_h = (oh + kDwTile - 1) / kDwTile;
    p.tiles_w = (ow + kDwTile - 1) / kDwTile;
    p.c_tiles = (d->c + kDwChannels - 1) / kDwChannels;
    p.in_h = (kDwTile - 1) * d->stride + (d->r - 1) * d->dilation + 1;
    p.in_w = (kDwTile - 1) * d->stride + (d->s - 1) * d->dilation + 1;
    p.x_words = ((fx.bits == 2 || fx.bits == 4 || fx.bits == 8) && ((int64_t)d->c * fx.bits) % 32 == 0) ? 1 : 0;
    const size_t smem = ((size_t)p.in_h * p.in_w + (size_t)d->r * d->s) * kDwChannels * sizeof(float);
    if (smem > 200 * 1024) return DYBIT_ERR_UNSUPPORTED;           // filter / stride too large for one staged patch
    const int64_t blocks = (int64_t)d->n * p.tiles_h * p.tiles_w * p.c_tiles;
    if (blocks > INT32_MAX) return DYBIT_ERR_UNSUPPORTED;
    DwTables tab;
    float vals[256];
    fill_table(fx, vals);
    for (int i = 0; i < 256; ++i) tab.x[i] = ldexpf(vals[i], mx - 1);
    fill_table(fw, vals);
    for (int i = 0; i < 256; ++i) tab.w[i] = ldexpf(vals[i], mw - 1);
    static bool configured[64] = {};
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(depthwise_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        configured[dev] = true;
    }
    launch_k(depthwise_kernel, dim3((unsigned)blocks), dim3(kDwThreads), smem, static_cast<cudaStream_t>(stream), p, tab);
    return launch_status();
}

}  // extern "C"

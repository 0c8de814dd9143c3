// Depth-wise convolution on DyBit-coded operands (the 3x3 layers of MobileNetV2, Section IV-A):
// every channel is filtered by its own r x s kernel, so there is no contraction a tensor core could
// carry -- r*s multiply-adds per output against 4 bytes written.  The kernel is bound by the fp32
// output stream; it decodes the packed codes itself, once per staged input element.
//
// Blocks are persistent and walk over tiles; one tile = one image, 16 x 8 output pixels, one slab of
// 32 channels:
//   1. the input patch the tile needs ((16-1)*stride + (r-1)*dilation + 1 rows, (8-1)*stride +
//      (s-1)*dilation + 1 columns, zeros outside the image) is decoded from the packed NHWC stream
//      into shared memory as fp32 integers value * 2^(m-1), channel innermost;
//   2. the slab's filters are decoded the same way, tap-major (once per slab);
//   3. warp w owns output rows 2w and 2w+1, lane l channel l: sixteen outputs per thread, each input
//      row held in registers across the filter columns and shared by both output rows; one fp32
//      FMA per tap (exact while the sums stay below 2^24, i.e. always for formats with at most 4
//      magnitude bits);
//   4. y = fmul_rn(sum, alpha): each warp writes 128 contiguous bytes per output pixel.
#pragma once

#include "dybit_common.cuh"
#include "dybit_host.cuh"

namespace dybit {

constexpr int kDwTile = 8;        // output columns per tile (= outputs per thread and row)
constexpr int kDwRowsPerWarp = 2;
constexpr int kDwWarps = 8;
constexpr int kDwTileRows = kDwWarps * kDwRowsPerWarp;
constexpr int kDwChannels = 32;   // channels per block (= lanes)
constexpr int kDwThreads = kDwWarps * 32;

struct DwParams {
    const uint8_t *X, *W;
    float *Y;
    const float *scale_x, *scale_w;
    double pow2;                  // alpha = (float)(scale_x * scale_w * pow2)
    int64_t ldw;
    int x_bits, w_bits;
    int N, H, Wd, C, R, S, OH, OW, stride, pad, dil;
    int tiles_h, tiles_w, c_tiles;
    int in_h, in_w;               // extent of the staged input patch
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

// The outputs of one thread (two rows of eight): RT x ST filter at stride STRIDE, dilation 1.  Every input
// row the two output rows touch is loaded into registers once.
template <int RT, int ST, int STRIDE>
__device__ __forceinline__ void dw_accumulate_fixed(const float *__restrict__ s_in, const float *__restrict__ s_w, int in_w,
                                                    int oy0, int lane, float (&acc)[kDwRowsPerWarp][kDwTile]) {
    constexpr int NC = (kDwTile - 1) * STRIDE + ST;
    constexpr int NR = (kDwRowsPerWarp - 1) * STRIDE + RT;
#pragma unroll
    for (int rr = 0; rr < NR; ++rr) {
        const float *row = s_in + (size_t)((oy0 * STRIDE + rr) * in_w) * kDwChannels + lane;
        float v[NC];
#pragma unroll
        for (int j = 0; j < NC; ++j) v[j] = row[j * kDwChannels];
#pragma unroll
        for (int q = 0; q < kDwRowsPerWarp; ++q) {
            const int r = rr - q * STRIDE;                       // filter row this input row meets for output row q
            if (r < 0 || r >= RT) continue;
#pragma unroll
            for (int s = 0; s < ST; ++s) {
                const float w = s_w[(r * ST + s) * kDwChannels + lane];
#pragma unroll
                for (int j = 0; j < kDwTile; ++j) acc[q][j] = fmaf(v[j * STRIDE + s], w, acc[q][j]);
            }
        }
    }
}

// XB = 2, 4, 8: X is read as whole 32-bit words (power-of-two width, word-aligned pixels); XB = 0: any width,
// code by code with byte loads.
template <int XB>
__global__ void __launch_bounds__(kDwThreads)
depthwise_kernel(const __grid_constant__ DwParams p, const __grid_constant__ DwTables tab) {
    extern __shared__ __align__(16) float dw_smem[];
    float *s_in = dw_smem;                                         // [in_h][in_w][32]
    float *s_w = dw_smem + (size_t)p.in_h * p.in_w * kDwChannels;  // [R*S][32]
    // word path: (row, column, word) of every decode item, the same for all tiles of a slab
    unsigned *s_item = reinterpret_cast<unsigned *>(s_w + (size_t)p.R * p.S * kDwChannels);
    __shared__ float s_lut_x[256], s_lut_w[256];
    pdl_enter();
    // the tables are read once per block (divergent reads of kernel parameters are slow)
    for (int i = threadIdx.x; i < 256; i += blockDim.x) {
        s_lut_x[i] = tab.x[i];
        s_lut_w[i] = tab.w[i];
    }
    const float alpha = (float)((double)__ldg(p.scale_x) * (double)__ldg(p.scale_w) * p.pow2);
    const int lane = threadIdx.x & 31, oy0 = (threadIdx.x >> 5) * kDwRowsPerWarp;
    const int spatial = p.tiles_h * p.tiles_w;
    const int per_slab = p.N * spatial;                         // tiles of one channel slab: slab index is the slowest
    const int total = per_slab * p.c_tiles;
    const int npix = p.in_h * p.in_w;
    int ct_loaded = -1;
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x) {
        const int ct = tile / per_slab;
        int b = tile - ct * per_slab;
        const int n = b / spatial;
        b -= n * spatial;
        const int th = b / p.tiles_w, tw = b - th * p.tiles_w;
        const int c0 = ct * kDwChannels;
        const int ih0 = th * kDwTileRows * p.stride - p.pad, iw0 = tw * kDwTile * p.stride - p.pad;
        constexpr int per_word = XB ? 32 / XB : 1;
        const int words = XB ? (min(kDwChannels, p.C - c0) * XB + 31) / 32 : 0;     // words of this slab per pixel
        __syncthreads();                                        // tables ready / previous tile's reads done

        if (ct != ct_loaded) {
            // filters of the slab, tap-major
            for (int i = threadIdx.x; i < p.R * p.S * kDwChannels; i += blockDim.x) {
                const int tap = i / kDwChannels, c = c0 + (i % kDwChannels);
                s_w[i] = c < p.C ? s_lut_w[stream_code(p.W + (int64_t)c * p.ldw, tap, p.w_bits)] : 0.0f;
            }
            if constexpr (XB != 0) {
                for (int i = threadIdx.x; i < npix * words; i += blockDim.x) {
                    const int pix = i / words, wd = i - pix * words;
                    const int iy = pix / p.in_w, ix = pix - iy * p.in_w;
                    s_item[i] = ((unsigned)iy << 20) | ((unsigned)ix << 8) | (unsigned)wd;
                }
                // channels of the slab past C (last slab only) that no word covers stay zero for all its tiles
                const int covered = words * per_word;
                if (covered < kDwChannels) {
                    const int rest = kDwChannels - covered;
                    for (int i = threadIdx.x; i < npix * rest; i += blockDim.x)
                        s_in[(size_t)(i / rest) * kDwChannels + covered + (i % rest)] = 0.0f;
                }
            }
            ct_loaded = ct;
            __syncthreads();
        }
        // input patch
        if constexpr (XB != 0) {
            // one 32-bit word of codes per thread and step: 32 / XB channels of one pixel
            constexpr unsigned mask = XB ? (1u << XB) - 1u : 0u;
            const int pixel_bytes = p.C * XB / 8;               // a multiple of 4 on this path
            const uint8_t *img = p.X + (int64_t)n * p.H * p.Wd * pixel_bytes + c0 * XB / 8;
            const bool whole = p.C - c0 >= kDwChannels;         // every word of the slab carries live channels only
            for (int i = threadIdx.x; i < npix * words; i += blockDim.x) {
                const unsigned item = s_item[i];
                const int iy = (int)(item >> 20), ix = (int)((item >> 8) & 0xfffu), wd = (int)(item & 0xffu);
                const int ih = ih0 + iy, iw = iw0 + ix;
                unsigned word = 0u;                               // code 0 decodes to 0 in every format
                if ((unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.Wd)
                    word = __ldg(reinterpret_cast<const unsigned *>(img + (ih * p.Wd + iw) * pixel_bytes) + wd);
                float *dst = s_in + (iy * p.in_w + ix) * kDwChannels + wd * per_word;
                if (whole) {
#pragma unroll
                    for (int k = 0; k < per_word; k += 4) {
                        float4 q;
                        q.x = s_lut_x[(word >> (XB * (k + 0) & 31)) & mask];
                        q.y = s_lut_x[(word >> (XB * (k + 1) & 31)) & mask];
                        q.z = s_lut_x[(word >> (XB * (k + 2) & 31)) & mask];
                        q.w = s_lut_x[(word >> (XB * (k + 3) & 31)) & mask];
                        *reinterpret_cast<float4 *>(dst + k) = q;
                    }
                } else {
                    const int live = min(per_word, p.C - c0 - wd * per_word);     // channels of this word that exist
                    for (int k = 0; k < per_word; ++k) dst[k] = k < live ? s_lut_x[(word >> (XB * k & 31)) & mask] : 0.0f;
                }
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

        float acc[kDwRowsPerWarp][kDwTile];
#pragma unroll
        for (int q = 0; q < kDwRowsPerWarp; ++q)
#pragma unroll
            for (int j = 0; j < kDwTile; ++j) acc[q][j] = 0.0f;
        if (p.R == 3 && p.S == 3 && p.dil == 1 && p.stride == 1) {
            dw_accumulate_fixed<3, 3, 1>(s_in, s_w, p.in_w, oy0, lane, acc);
        } else if (p.R == 3 && p.S == 3 && p.dil == 1 && p.stride == 2) {
            dw_accumulate_fixed<3, 3, 2>(s_in, s_w, p.in_w, oy0, lane, acc);
        } else {
            for (int r = 0; r < p.R; ++r) {
                for (int s = 0; s < p.S; ++s) {
                    const float w = s_w[(r * p.S + s) * kDwChannels + lane];
#pragma unroll
                    for (int q = 0; q < kDwRowsPerWarp; ++q) {
                        const float *row = s_in + (size_t)(((oy0 + q) * p.stride + r * p.dil) * p.in_w) * kDwChannels + lane;
#pragma unroll
                        for (int j = 0; j < kDwTile; ++j)
                            acc[q][j] = fmaf(row[(j * p.stride + s * p.dil) * kDwChannels], w, acc[q][j]);
                    }
                }
            }
        }
        const int c = c0 + lane;
        const int ow_left = p.OW - tw * kDwTile;                // columns of this tile inside the image
#pragma unroll
        for (int q = 0; q < kDwRowsPerWarp; ++q) {
            const int oh = th * kDwTileRows + oy0 + q;
            if (oh < p.OH && c < p.C) {
                float *yrow = p.Y + (((int64_t)n * p.OH + oh) * p.OW + (int64_t)tw * kDwTile) * p.C + c;
                if (ow_left >= kDwTile) {
#pragma unroll
                    for (int j = 0; j < kDwTile; ++j) __stcs(yrow + j * p.C, __fmul_rn(acc[q][j], alpha));
                } else {
#pragma unroll
                    for (int j = 0; j < kDwTile; ++j)
                        if (j < ow_left) __stcs(yrow + j * p.C, __fmul_rn(acc[q][j], alpha));
                }
            }
        }
    }
}

template <int XB>
static dybit_status launch_depthwise(const DwParams &p, const DwTables &tab, size_t smem, int64_t tiles, cudaStream_t s) {
    static std::atomic<bool> configured[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(depthwise_kernel<XB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        configured[dev] = true;
    }
    // persistent blocks: exactly as many as are resident at once, each walking over tiles
    int per_sm = 1;
    DYBIT_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, depthwise_kernel<XB>, kDwThreads, smem));
    if (per_sm < 1) per_sm = 1;
    const int64_t grid = tiles < (int64_t)sm_count() * per_sm ? tiles : (int64_t)sm_count() * per_sm;
    launch_k(depthwise_kernel<XB>, dim3((unsigned)grid), dim3(kDwThreads), smem, s, p, tab);
    return launch_status();
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
    p.N = d->n; p.H = d->h; p.Wd = d->w; p.C = d->c; p.R = d->r; p.S = d->s;
    p.OH = oh; p.OW = ow; p.stride = d->stride; p.pad = d->pad; p.dil = d->dilation;
    p.tiles_h = (oh + kDwTileRows - 1) / kDwTileRows;
    p.tiles_w = (ow + kDwTile - 1) / kDwTile;
    p.c_tiles = (d->c + kDwChannels - 1) / kDwChannels;
    p.in_h = (kDwTileRows - 1) * d->stride + (d->r - 1) * d->dilation + 1;
    p.in_w = (kDwTile - 1) * d->stride + (d->s - 1) * d->dilation + 1;
    const bool by_words = (fx.bits == 2 || fx.bits == 4 || fx.bits == 8) && ((int64_t)d->c * fx.bits) % 32 == 0 &&
                          p.in_h < 4096 && p.in_w < 4096;
    const size_t smem = ((size_t)p.in_h * p.in_w + (size_t)d->r * d->s) * kDwChannels * sizeof(float) +
                        (by_words ? (size_t)p.in_h * p.in_w * fx.bits * sizeof(unsigned) : 0);   // + decode items
    if (smem > 200 * 1024) return DYBIT_ERR_UNSUPPORTED;           // filter / stride too large for one staged patch
    if ((int64_t)d->h * d->w * d->c * fx.bits / 8 > INT32_MAX || (int64_t)ow * d->c * 8 > INT32_MAX)
        return DYBIT_ERR_UNSUPPORTED;                              // offsets inside one image are 32-bit
    const int64_t tiles = (int64_t)d->n * p.tiles_h * p.tiles_w * p.c_tiles;
    if (tiles > INT32_MAX) return DYBIT_ERR_UNSUPPORTED;
    DwTables tab;
    float vals[256];
    fill_table(fx, vals);
    for (int i = 0; i < 256; ++i) tab.x[i] = ldexpf(vals[i], mx - 1);
    fill_table(fw, vals);
    for (int i = 0; i < 256; ++i) tab.w[i] = ldexpf(vals[i], mw - 1);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!by_words) return launch_depthwise<0>(p, tab, smem, tiles, s);
    switch (fx.bits) {
        case 2: return launch_depthwise<2>(p, tab, smem, tiles, s);
        case 4: return launch_depthwise<4>(p, tab, smem, tiles, s);
        default: return launch_depthwise<8>(p, tab, smem, tiles, s);
    }
}

}  // extern "C"

// GEMM / implicit-GEMM convolution on DyBit-coded operands.
//
// Two steps per call:
//   1. expand: packed codes -> the container type (int8 / e4m3 / bf16) through
//      the enumerated value table, written once into caller workspace
//      (O(MK + NK) work, HBM-bound);
//   2. a persistent, warp-specialised tcgen05 GEMM on the expanded operands:
//      TMA (128-byte swizzle) -> shared-memory ring -> tcgen05.mma with the
//      accumulator in tensor memory -> epilogue warps read TMEM, apply alpha
//      and store fp32 (and the raw int32 sum when asked).
// The convolution is the same kernel with the A tile gathered straight from the
// expanded NHWC activation (im2col addressing, zero fill for padding taps).
#pragma once

#include <thread>

#include "dybit_common.cuh"
#include "dybit_host.cuh"
#include "dybit_quantize.cuh"
#include "dybit_sm100.cuh"

namespace dybit {

using namespace sm100;

// ------------------------------------------------------------------ expand kernels

struct ElemTable {
    uint16_t v[256];   // container bit pattern of each code's value (low byte used for 1-byte containers)
};

// bf16 / e4m3 / int8 bit patterns of a value that is known to be exactly representable.
static uint16_t to_bf16_bits(float v) {
    uint32_t u;
    memcpy(&u, &v, 4);
    return (uint16_t)(u >> 16);
}

static uint8_t to_e4m3_bits(float v) {
    if (v == 0.0f) return 0;
    uint8_t sign = v < 0 ? 0x80 : 0;
    float a = fabsf(v);
    int e;
    float fr = frexpf(a, &e);            // a = fr * 2^e, fr in [0.5,1)  ->  1.f * 2^(e-1)
    int exp = e - 1;
    if (exp >= -6) {
        int mant = (int)lrintf(ldexpf(fr, 4)) - 8;          // 3 fraction bits
        return sign | (uint8_t)(((exp + 7) << 3) | mant);
    }
    int mant = (int)lrintf(ldexpf(a, 9));                   // subnormal: multiples of 2^-9
    return sign | (uint8_t)mant;
}

static ElemTable make_elem_table_uncached(dybit_fmt f, dybit_container cont, int int_exp) {
    float tab[256];
    fill_table(f, tab);
    ElemTable t;
    for (int c = 0; c < 256; ++c) {
        switch (cont) {
            case DYBIT_CONTAINER_I8: t.v[c] = (uint16_t)(uint8_t)(int8_t)lrintf(ldexpf(tab[c], int_exp)); break;
            case DYBIT_CONTAINER_E4M3: t.v[c] = to_e4m3_bits(tab[c]); break;
            default: t.v[c] = to_bf16_bits(tab[c]); break;
        }
    }
    return t;
}

// One table per (format, container); the int8 rescale exponent is a function of the format alone.
static const ElemTable &make_elem_table(dybit_fmt f, dybit_container cont, int int_exp) {
    struct Entry {
        std::atomic<int> state{0};
        ElemTable table;
    };
    static Entry cache[14][3];
    Entry &e = cache[fmt_index(f)][(int)cont];
    if (e.state.load(std::memory_order_acquire) != 2) {
        int expected = 0;
        if (e.state.compare_exchange_strong(expected, 1)) {
            e.table = make_elem_table_uncached(f, cont, int_exp);
            e.state.store(2, std::memory_order_release);
        } else {
            // another thread is filling this entry (a few microseconds of host work): wait for it
            while (e.state.load(std::memory_order_acquire) != 2) std::this_thread::yield();
        }
    }
    return e.table;
}

// Rows of packed codes -> rows of container elements.  A warp expands 1024 codes at a time and keeps the packed
// vectors of two such chunks in flight.
template <int BITS, int ELEM>
__global__ void __launch_bounds__(kStreamThreads)
expand_rows_kernel(const uint8_t *__restrict__ packed, int64_t rows, int64_t in_stride, int64_t cols,
                   uint8_t *__restrict__ out, int64_t out_stride, const __grid_constant__ ElemTable table) {
    __shared__ uint16_t s_lut[256];
    __shared__ __align__(16) unsigned s_words[kWarpsPerBlock][2][32 * BITS];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = table.v[i];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_enter();
    constexpr int kChunkBytes = kChunkCodes * BITS / 8;
    constexpr int kChunkVecs = kChunkBytes / 16;
    const int64_t chunks_per_row = (cols + kChunkCodes - 1) / kChunkCodes;
    const int64_t items = rows * chunks_per_row;
    const int64_t in_row_bytes = ((cols * BITS + 7) / 8 + 15) / 16 * 16;
    const int64_t stride = (int64_t)gridDim.x * kWarpsPerBlock;
    for (int64_t item0 = (int64_t)blockIdx.x * kWarpsPerBlock + warp; item0 < items; item0 += 2 * stride) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int64_t item = item0 + u * stride;
            if (item >= items) continue;
            const int64_t row = item / chunks_per_row, chunk = item - row * chunks_per_row;
            const int nvec = (int)min((int64_t)kChunkVecs, (in_row_bytes - chunk * kChunkBytes) / 16);
            const uint4 *src = reinterpret_cast<const uint4 *>(packed + row * in_stride + chunk * kChunkBytes);
            uint4 *s4 = reinterpret_cast<uint4 *>(&s_words[warp][u][0]);
            for (int i = lane; i < kChunkVecs; i += 32) s4[i] = (i < nvec) ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int64_t item = item0 + u * stride;
            if (item >= items) continue;
            const int64_t row = item / chunks_per_row, chunk = item - row * chunks_per_row;
            const int64_t c0 = chunk * kChunkCodes;
            const int valid = (int)min((int64_t)kChunkCodes, cols - c0);
            unsigned w[BITS], cw[8];
#pragma unroll
            for (int i = 0; i < BITS; ++i) w[i] = s_words[warp][u][lane * BITS + i];
            unpack32<BITS>(w, cw);
            uint8_t *dst = out + row * out_stride + (c0 + lane * 32) * ELEM;
            if constexpr (ELEM == 1) {
                unsigned o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    o[i] = (unsigned)(s_lut[cw[i] & 0xffu] & 0xffu) | ((unsigned)(s_lut[(cw[i] >> 8) & 0xffu] & 0xffu) << 8) |
                           ((unsigned)(s_lut[(cw[i] >> 16) & 0xffu] & 0xffu) << 16) |
                           ((unsigned)(s_lut[cw[i] >> 24] & 0xffu) << 24);
                }
                if (lane * 32 < valid) reinterpret_cast<uint4 *>(dst)[0] = make_uint4(o[0], o[1], o[2], o[3]);
                if (lane * 32 + 16 < valid) reinterpret_cast<uint4 *>(dst)[1] = make_uint4(o[4], o[5], o[6], o[7]);
            } else {
                unsigned o[16];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    o[2 * i] = (unsigned)s_lut[cw[i] & 0xffu] | ((unsigned)s_lut[(cw[i] >> 8) & 0xffu] << 16);
                    o[2 * i + 1] = (unsigned)s_lut[(cw[i] >> 16) & 0xffu] | ((unsigned)s_lut[cw[i] >> 24] << 16);
                }
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    if (lane * 32 + v * 8 < valid)
                        reinterpret_cast<uint4 *>(dst)[v] = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
            }
        }
        __syncwarp();
    }
}

// 4-bit codes -> 1-byte container elements without shared memory.  A 32-bit word holds eight codes; the
// byte-permute unit looks four of them up at once in a 16-entry table kept in four registers.  A selector
// nibble with its top bit set makes prmt replicate the selected byte's sign bit, which is 0x00 for the
// non-negative bytes stored here, so "lookup in the low half with the raw nibbles" and "lookup in the high
// half with the top bits flipped" each yield 0 for the codes that belong to the other half.
//   neg_high = false: the table's entries are used as they are (all 16 values non-negative): result = lo | hi
//   neg_high = true : entries 8..15 hold MAGNITUDES of negative values: result = lo - hi, byte-wise
// Two independent operands (jobs) can share one launch.
struct Expand4Job {
    const uint8_t *packed;
    uint8_t *out;
    int64_t rows, in_stride, out_stride;
    int64_t vecs_per_row;      // 16-byte input vectors (32 codes) per row
    unsigned tab[4];           // 16 table bytes
    int neg_high;
};

// prmt in its generic form: selector nibble bits 0-2 pick one of the eight source bytes, bit 3 asks
// for that byte's sign bit replicated instead of the byte (the __byte_perm intrinsic drops bit 3).
__device__ __forceinline__ unsigned prmt_generic(unsigned a, unsigned b, unsigned sel) {
    unsigned d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__device__ __forceinline__ unsigned expand4_lookup(unsigned sel, const unsigned (&t)[4], bool neg_high) {
    const unsigned lo = prmt_generic(t[0], t[1], sel);
    const unsigned hi = prmt_generic(t[2], t[3], sel ^ 0x8888u);
    // byte-wise lo - hi: never both non-zero; the 0x80 guard bits stop borrows between bytes
    return neg_high ? (((lo | 0x80808080u) - hi) ^ 0x80808080u) : (lo | hi);
}

__global__ void __launch_bounds__(256) expand4_kernel(const Expand4Job j0, const Expand4Job j1, int64_t vecs0) {
    pdl_enter();
    const int64_t total = vecs0 + j1.rows * j1.vecs_per_row;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    // two 16-byte vectors of codes in flight per thread and round trip
    for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < total; i0 += 2 * stride) {
        uint4 w[2];
        uint4 *dst[2];
        bool ng[2];
        unsigned t[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int64_t i = i0 + u * stride;
            dst[u] = nullptr;
            if (i >= total) continue;
            const bool first = i < vecs0;
            const Expand4Job &j = first ? j0 : j1;
            const int64_t v = first ? i : i - vecs0;
            // (rows of up to 2^31 vectors: one 64-bit division only when the index does not fit 32 bits)
            int64_t row, col;
            if (v < ((int64_t)1 << 32) && j.vecs_per_row < ((int64_t)1 << 32)) {
                const unsigned r32 = (unsigned)v / (unsigned)j.vecs_per_row;
                row = r32;
                col = (int64_t)((unsigned)v - r32 * (unsigned)j.vecs_per_row);
            } else {
                row = v / j.vecs_per_row;
                col = v - row * j.vecs_per_row;
            }
            w[u] = __ldg(reinterpret_cast<const uint4 *>(j.packed + row * j.in_stride) + col);
#pragma unroll
            for (int k = 0; k < 4; ++k) t[u][k] = j.tab[k];
            ng[u] = j.neg_high != 0;
            if (DYBIT_CHECK(row < j.rows && col * 32 + 32 <= (j.rows > 1 ? j.out_stride : j.vecs_per_row * 32), 0x23))
                dst[u] = reinterpret_cast<uint4 *>(j.out + row * j.out_stride + col * 32);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (dst[u] == nullptr) continue;
            uint4 o0, o1;
            o0.x = expand4_lookup(w[u].x, t[u], ng[u]); o0.y = expand4_lookup(w[u].x >> 16, t[u], ng[u]);
            o0.z = expand4_lookup(w[u].y, t[u], ng[u]); o0.w = expand4_lookup(w[u].y >> 16, t[u], ng[u]);
            o1.x = expand4_lookup(w[u].z, t[u], ng[u]); o1.y = expand4_lookup(w[u].z >> 16, t[u], ng[u]);
            o1.z = expand4_lookup(w[u].w, t[u], ng[u]); o1.w = expand4_lookup(w[u].w >> 16, t[u], ng[u]);
            dst[u][0] = o0;
            dst[u][1] = o1;
        }
    }
}

// Generic (slow) expand with channel padding: output row = taps x cp elements, where tap t
// takes codes [t*c, t*c + c) of the input row's bit stream and pads channels c..cp-1 with 0.
// One thread writes one 16-byte output chunk.
__global__ void expand_pad_kernel(const uint8_t *__restrict__ packed, int bits, int64_t rows, int64_t in_stride,
                                  int64_t taps, int c, int cp, int elem, uint8_t *__restrict__ out,
                                  int64_t out_stride, const __grid_constant__ ElemTable table) {
    const int per_chunk = 16 / elem;
    const int64_t chunks_per_tap = cp / per_chunk;
    pdl_enter();
    const int64_t total = rows * taps * chunks_per_tap;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t g = idx % chunks_per_tap;
        const int64_t t = (idx / chunks_per_tap) % taps;
        const int64_t row = idx / (chunks_per_tap * taps);
        const uint8_t *src = packed + row * in_stride;
        unsigned o[4] = {0, 0, 0, 0};
        for (int e = 0; e < per_chunk; ++e) {
            const int ch = (int)g * per_chunk + e;
            unsigned code = 0;
            if (ch < c) {
                const int64_t bit = (t * c + ch) * bits;
                const int sh = (int)(bit & 7);
                unsigned two = src[bit >> 3];
                if (sh + bits > 8) two |= (unsigned)src[(bit >> 3) + 1] << 8;
                code = (two >> sh) & ((1u << bits) - 1u);
            }
            const unsigned v = table.v[code];
            if (elem == 1) o[e >> 2] |= (v & 0xffu) << ((e & 3) * 8);
            else o[e >> 1] |= v << ((e & 1) * 16);
        }
        uint8_t *dst = out + row * out_stride + (t * cp + g * per_chunk) * elem;
        *reinterpret_cast<uint4 *>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// ------------------------------------------------------------------ quantize + expand in one launch

// A weight matrix to expand alongside: rows of `cols` container elements from rows of packed codes.
struct FusedWeights {
    const uint8_t *packed;
    int bits;
    int64_t rows, in_stride, cols;
    uint8_t *out;
    int64_t out_stride;
    int use4;                 // 1: job4 describes the same rows for the 4-bit register-table expansion
    Expand4Job job4;
    int pix_c, pix_r, pix_s;  // pix_c > 0: filter rows of 8 taps x 4 bytes instead (see expand_weights_pix4)
    int s2d;                  // 1 (with pix_c/r/s set): space-to-depth filter layout instead (see expand_weights_s2d)
    int s2d_lo_r, s2d_lo_s, s2d_pad, s2d_rp;
};

// Geometry of the 2 x 2 space-to-depth rearrangement of a stride-2 convolution's input (ConvMode kConvS2D).
// Rearranged pixel (hh, ww) holds input pixels (2hh + dy, 2ww + dx), dy, dx in {0, 1}, C bytes each at byte
// (2dy + dx) * C; input row 2*oh - pad + r lies in rearranged row oh + lo_r + r' with r' = floor((r - pad) / 2) - lo_r.
struct S2dGeom {
    int Hs, Ws;               // rearranged image: H / 2 x W / 2 pixels of 16 bytes
    int P;                    // pixels per stored row: padL zero pixels, Ws pixels, 3 zero pixels
    int padL;                 // = -lo_s
    int lo_r, lo_s;           // first rearranged row / column of a window, relative to the output pixel
    int Rp, Sp;               // rearranged filter rows / columns (both <= 4)
};

// Where quantize_expand_kernel / expand_pix4_kernel put the container bytes of a pixel with <= 4 one-byte channels:
// one 32-bit word per pixel in NHW order (s2d = 0), or the space-to-depth image (s2d = 1).
struct PixLayout {
    int c;                    // channels per pixel; 0: not a few-channel layout at all
    int s2d;
    int H, W, Hs, P, padL;
};

// Space-to-depth image: where the channel bytes of input pixel `px` (NHW index) go.
// (pixel counts fit 32 bits: the host checks it before it takes this lowering)
__device__ __forceinline__ uint8_t *s2d_pixel_addr(uint8_t *xs, const PixLayout &pl, int64_t px) {
    const unsigned hw = (unsigned)(pl.H * pl.W);
    const unsigned img = (unsigned)px / hw, rem = (unsigned)px - img * hw;
    const unsigned h = rem / (unsigned)pl.W, w = rem - h * (unsigned)pl.W;
    return xs + ((((int64_t)(img * (unsigned)pl.Hs + (h >> 1)) * pl.P + (w >> 1) + pl.padL) << 4) + ((h & 1) * 2 + (w & 1)) * pl.c);
}

// The zero bytes pixel `px` is responsible for: the unused tail of its 16-byte block (the block's last pixel writes
// it) and the padding pixels of its stored row (the first and last pixel of every even input row write them).
__device__ __forceinline__ void s2d_pixel_duties(uint8_t *xs, const PixLayout &pl, int64_t px) {
    const unsigned hw = (unsigned)(pl.H * pl.W);
    const unsigned img = (unsigned)px / hw, rem = (unsigned)px - img * hw;
    const int h = (int)(rem / (unsigned)pl.W), w = (int)(rem - (unsigned)h * (unsigned)pl.W);
    uint8_t *row = xs + (((int64_t)(img * (unsigned)pl.Hs + ((unsigned)h >> 1)) * pl.P) << 4);
    if ((h & 1) && (w & 1)) {
        uint8_t *blk = row + (((w >> 1) + pl.padL) << 4);
        for (int b = 4 * pl.c; b < 16; ++b) blk[b] = 0;
    }
    if (!(h & 1)) {
        if (w == 0)
            for (int i = 0; i < pl.padL; ++i) reinterpret_cast<uint4 *>(row)[i] = make_uint4(0, 0, 0, 0);
        if (w == pl.W - 1)
            for (int i = 0; i < 3; ++i) reinterpret_cast<uint4 *>(row)[pl.padL + (pl.W >> 1) + i] = make_uint4(0, 0, 0, 0);
    }
}

__device__ __forceinline__ void s2d_store_pixel(uint8_t *xs, const PixLayout &pl, int64_t px, unsigned word) {
    uint8_t *dst = s2d_pixel_addr(xs, pl, px);
    for (int b = 0; b < pl.c; ++b) dst[b] = (uint8_t)(word >> (8 * b));
    s2d_pixel_duties(xs, pl, px);
}

// The activation's own 16-entry table for the register-table expansion of 4-bit codes (see expand4_lookup); use = 0
// keeps the shared-memory table.
struct XTab4 {
    unsigned tab[4];
    int use, neg_high;
};

// Weights for the few-channel lowering (ConvMode kConvPix4): row n of the output holds, for each filter row r,
// eight taps of four bytes: tap s < S carries its C <= 4 one-byte elements, everything else is zero; rows are
// padded with zeros to out_stride.  Thread `idx` writes one 16-byte chunk (four taps).
__device__ __forceinline__ void expand_weights_pix4(const FusedWeights &wj, const uint16_t *s_lut, int64_t idx) {
    const int64_t chunks_per_row = wj.out_stride / 16;
    const int64_t row = idx / chunks_per_row;
    const int g = (int)(idx - row * chunks_per_row);
    const int r = g >> 1, s0 = (g & 1) * 4;
    const uint8_t *src = wj.packed + row * wj.in_stride;
    const unsigned mask = (1u << wj.bits) - 1u;
    unsigned o[4] = {0, 0, 0, 0};
    for (int t = 0; t < 4; ++t) {
        const int s = s0 + t;
        if (r >= wj.pix_r || s >= wj.pix_s) continue;
        for (int c = 0; c < wj.pix_c; ++c) {
            const int64_t bit = (int64_t)((r * wj.pix_s + s) * wj.pix_c + c) * wj.bits;
            const int sh = (int)(bit & 7);
            unsigned two = __ldg(src + (bit >> 3));
            if (sh + wj.bits > 8) two |= (unsigned)__ldg(src + (bit >> 3) + 1) << 8;
            o[t] |= (unsigned)(s_lut[(two >> sh) & mask] & 0xffu) << (8 * c);
        }
    }
    *reinterpret_cast<uint4 *>(wj.out + row * wj.out_stride + g * 16) = make_uint4(o[0], o[1], o[2], o[3]);
}

// Weights for the space-to-depth lowering (ConvMode kConvS2D): row n of the output holds, for each rearranged filter
// row r', four rearranged taps s' of 16 bytes; byte (2dy + dx) * C + c of tap (r', s') is the weight of the original
// tap r = 2 (r' + lo_r) + dy + pad, s = 2 (s' + lo_s) + dx + pad, channel c, or zero when that tap does not exist.
// Thread `idx` writes one 16-byte chunk (one rearranged tap); chunks past the last filter row are zero.
__device__ __forceinline__ void expand_weights_s2d(const FusedWeights &wj, const uint16_t *s_lut, int64_t idx) {
    const int64_t chunks_per_row = wj.out_stride / 16;
    const int64_t row = idx / chunks_per_row;
    const int g = (int)(idx - row * chunks_per_row);
    const int rp = g >> 2, sp = g & 3;
    const uint8_t *src = wj.packed + row * wj.in_stride;
    const unsigned mask = (1u << wj.bits) - 1u;
    unsigned o[4] = {0, 0, 0, 0};
    if (rp < wj.s2d_rp) {
        for (int dy = 0; dy < 2; ++dy) {
            for (int dx = 0; dx < 2; ++dx) {
                const int r = 2 * (rp + wj.s2d_lo_r) + dy + wj.s2d_pad, s = 2 * (sp + wj.s2d_lo_s) + dx + wj.s2d_pad;
                if (r < 0 || r >= wj.pix_r || s < 0 || s >= wj.pix_s) continue;
                for (int c = 0; c < wj.pix_c; ++c) {
                    const int64_t bit = (int64_t)((r * wj.pix_s + s) * wj.pix_c + c) * wj.bits;
                    const int sh = (int)(bit & 7);
                    unsigned two = __ldg(src + (bit >> 3));
                    if (sh + wj.bits > 8) two |= (unsigned)__ldg(src + (bit >> 3) + 1) << 8;
                    const int byte = (dy * 2 + dx) * wj.pix_c + c;
                    o[byte >> 2] |= (unsigned)(s_lut[(two >> sh) & mask] & 0xffu) << (8 * (byte & 3));
                }
            }
        }
    }
    *reinterpret_cast<uint4 *>(wj.out + row * wj.out_stride + g * 16) = make_uint4(o[0], o[1], o[2], o[3]);
}

// fp32 activation -> packed codes AND their container elements, plus the layer's weights expanded by the
// last blocks of the same grid: what dybit_quantize_pack followed by the expand launch of dybit_conv2d
// compute, in one launch instead of two.  The activation is one flat run of n elements whose expanded
// layout is the code order itself (channels a multiple of 16).  Blocks [0, x_blocks) take the activation,
// a warp 1024 elements at a time exactly as quantize_pack_kernel does; the others the weights, one
// 16-byte output chunk per thread.  With `partials` the max-abs reduction is finished here as well (see
// scale_from_partials) and block 0 stores the {scale, 1/scale} pair in scale_out.
// What one activation, and the weights of its layer, need from quantize_expand_kernel.
struct QeArgs {
    const float *x;
    int64_t n;
    const float *scale;
    uint8_t *packed;
    int64_t packed_bytes;
    uint8_t *xe;
    int64_t xe_bytes;
    FusedWeights wj;
    int x_blocks;                    // blocks [0, x_blocks) of the layer's share take the activation, the rest the weights
    const unsigned *partials;
    int n_partials, m;
    float *scale_out;
    PixLayout pl;
};

// Block `bid` of the `nblk` blocks that work on the layer described by `a`.
template <int BITS, bool SIGNED, int ELEM>
__device__ __forceinline__ void quantize_expand_body(const QeArgs &a, const ElemTable &tx, const ElemTable &tw, const XTab4 &xt,
                                                     const int bid, const int nblk) {
    const float *__restrict__ x = a.x;
    const int64_t n = a.n;
    const float *__restrict__ scale = a.scale;
    uint8_t *__restrict__ packed = a.packed;
    const int64_t packed_bytes = a.packed_bytes;
    uint8_t *__restrict__ xe = a.xe;
    const int64_t xe_bytes = a.xe_bytes;
    const FusedWeights &wj = a.wj;
    const int x_blocks = a.x_blocks;
    const unsigned *__restrict__ partials = a.partials;
    const int n_partials = a.n_partials, m = a.m;
    float *__restrict__ scale_out = a.scale_out;
    const PixLayout &pl = a.pl;
    const int pix_c = pl.c;
    __shared__ __align__(16) unsigned s_codes[kWarpsPerBlock][kChunkCodes / 4];
    __shared__ __align__(16) unsigned s_words[kWarpsPerBlock][32 * BITS];
    __shared__ uint16_t s_lut[256];
    const bool weights = bid >= x_blocks;
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = weights ? tw.v[i] : tx.v[i];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    constexpr int kChunkBytes = kChunkCodes * BITS / 8;
    constexpr int kChunkVecs = kChunkBytes / 16;
    const int64_t items = (packed_bytes + kChunkBytes - 1) / kChunkBytes;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
    const int64_t first_item = (int64_t)bid * kWarpsPerBlock + warp;
    float4 v[8];
    auto load_item = [&](int64_t item) {
        const int64_t c0 = item * kChunkCodes;
        const float *src = x + c0;
        const int64_t valid = min((int64_t)kChunkCodes, max((int64_t)0, n - c0));
        if (valid == kChunkCodes && vec_ok) {
            const float4 *s4 = reinterpret_cast<const float4 *>(src);
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __ldcs(s4 + j * 32 + lane);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t i0 = j * 128 + lane * 4;
                v[j].x = (i0 + 0 < valid) ? src[i0 + 0] : 0.0f;
                v[j].y = (i0 + 1 < valid) ? src[i0 + 1] : 0.0f;
                v[j].z = (i0 + 2 < valid) ? src[i0 + 2] : 0.0f;
                v[j].w = (i0 + 3 < valid) ? src[i0 + 3] : 0.0f;
            }
        }
    };
    // With `partials` the kernel in front of this one is the max-abs pass over the same x, which only reads it: x
    // itself was complete before that pass began, so the first chunk can be fetched while it is still draining.
    const bool early = partials != nullptr && !weights && first_item < items;
    if (early) load_item(first_item);
    pdl_enter();
    if (weights) {
        if (wj.pix_c > 0) {
            const int64_t total = wj.rows * (wj.out_stride / 16);
            for (int64_t idx = (int64_t)(bid - x_blocks) * blockDim.x + threadIdx.x; idx < total;
                 idx += (int64_t)(nblk - x_blocks) * blockDim.x) {
                if (wj.s2d) expand_weights_s2d(wj, s_lut, idx);
                else expand_weights_pix4(wj, s_lut, idx);
            }
            return;
        }
        if (wj.use4) {
            // 4-bit codes through the 16-entry register table: one 16-byte vector of codes per step
            const Expand4Job &j = wj.job4;
            const int64_t total = j.rows * j.vecs_per_row;
            const unsigned t[4] = {j.tab[0], j.tab[1], j.tab[2], j.tab[3]};
            const bool ng = j.neg_high != 0;
            for (int64_t i = (int64_t)(bid - x_blocks) * blockDim.x + threadIdx.x; i < total;
                 i += (int64_t)(nblk - x_blocks) * blockDim.x) {
                const int64_t row = i / j.vecs_per_row, col = i - row * j.vecs_per_row;
                const uint4 w = __ldg(reinterpret_cast<const uint4 *>(j.packed + row * j.in_stride) + col);
                uint4 o0, o1;
                o0.x = expand4_lookup(w.x, t, ng); o0.y = expand4_lookup(w.x >> 16, t, ng);
                o0.z = expand4_lookup(w.y, t, ng); o0.w = expand4_lookup(w.y >> 16, t, ng);
                o1.x = expand4_lookup(w.z, t, ng); o1.y = expand4_lookup(w.z >> 16, t, ng);
                o1.z = expand4_lookup(w.w, t, ng); o1.w = expand4_lookup(w.w >> 16, t, ng);
                uint4 *dst = reinterpret_cast<uint4 *>(j.out + row * j.out_stride + col * 32);
                dst[0] = o0;
                dst[1] = o1;
            }
            return;
        }
        constexpr int per_chunk = 16 / ELEM;
        const int64_t chunks_per_row = wj.cols / per_chunk;
        const int64_t total = wj.rows * chunks_per_row;
        const unsigned mask = (1u << wj.bits) - 1u;
        for (int64_t idx = (int64_t)(bid - x_blocks) * blockDim.x + threadIdx.x; idx < total;
             idx += (int64_t)(nblk - x_blocks) * blockDim.x) {
            const int64_t row = idx / chunks_per_row, g = idx - row * chunks_per_row;
            const uint8_t *src = wj.packed + row * wj.in_stride;
            unsigned o[4] = {0, 0, 0, 0};
#pragma unroll
            for (int e = 0; e < per_chunk; ++e) {
                const int64_t bit = (g * per_chunk + e) * wj.bits;
                const int sh = (int)(bit & 7);
                unsigned two = __ldg(src + (bit >> 3));
                if (sh + wj.bits > 8) two |= (unsigned)__ldg(src + (bit >> 3) + 1) << 8;
                const unsigned v = s_lut[(two >> sh) & mask];
                if (ELEM == 1) o[e >> 2] |= (v & 0xffu) << ((e & 3) * 8);
                else o[e >> 1] |= v << ((e & 1) * 16);
            }
            *reinterpret_cast<uint4 *>(wj.out + row * wj.out_stride + g * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        }
        return;
    }
    // the scale is either there already, or made here from the per-block maxima the preceding absmax launch left
    const float inv = partials ? scale_from_partials(partials, n_partials, m, scale_out, bid == 0) : __ldg(scale + 1);
    for (int64_t item = first_item; item < items; item += (int64_t)x_blocks * kWarpsPerBlock) {
        const int64_t c0 = item * kChunkCodes;
        const int nvec = (int)min((int64_t)kChunkVecs, (packed_bytes - item * kChunkBytes) / 16);
        if (!(early && item == first_item)) load_item(item);
#pragma unroll
        for (int j = 0; j < 8; ++j) s_codes[warp][j * 32 + lane] = encode4<BITS, SIGNED>(v[j], inv);
        __syncwarp();
        // lane takes codes [32*lane, 32*lane + 32)
        unsigned cw[8];
        {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(&s_codes[warp][lane * 8]);
            const int first = (lane >> 2) & 1;
            uint4 a = s4[first], b = s4[first ^ 1];
            if (first) { uint4 t = a; a = b; b = t; }
            cw[0] = a.x; cw[1] = a.y; cw[2] = a.z; cw[3] = a.w;
            cw[4] = b.x; cw[5] = b.y; cw[6] = b.z; cw[7] = b.w;
        }
        // container elements of the same 32 codes
        {
            const int64_t off = (c0 + lane * 32) * ELEM;
            if constexpr (ELEM == 1) {
                unsigned o[8];
                bool looked_up = false;
                if constexpr (BITS == 4) {
                    if (xt.use) {
                        // eight codes per packed word -> two words of elements, through the table held in registers
                        unsigned w4[4];
                        pack32<4>(cw, w4);
                        const unsigned t4[4] = {xt.tab[0], xt.tab[1], xt.tab[2], xt.tab[3]};
                        const bool ng = xt.neg_high != 0;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            o[2 * i] = expand4_lookup(w4[i], t4, ng);
                            o[2 * i + 1] = expand4_lookup(w4[i] >> 16, t4, ng);
                        }
                        looked_up = true;
                    }
                }
                if (!looked_up) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        o[i] = (unsigned)(s_lut[cw[i] & 0xffu] & 0xffu) | ((unsigned)(s_lut[(cw[i] >> 8) & 0xffu] & 0xffu) << 8) |
                               ((unsigned)(s_lut[(cw[i] >> 16) & 0xffu] & 0xffu) << 16) | ((unsigned)(s_lut[cw[i] >> 24] & 0xffu) << 24);
                }
                if (pix_c > 0) {
                    // pixels of pix_c < 4 one-byte elements, each padded to a 32-bit word: the chunk's 1024 bytes go
                    // back to shared memory in element order, lanes then assemble whole pixels; the (at most two)
                    // pixels that straddle the chunk's ends are completed byte by byte by both chunks involved
                    __syncwarp();
                    uint4 *mine = reinterpret_cast<uint4 *>(&s_codes[warp][lane * 8]);
                    mine[0] = make_uint4(o[0], o[1], o[2], o[3]);
                    mine[1] = make_uint4(o[4], o[5], o[6], o[7]);
                    __syncwarp();
                    const uint8_t *sb = reinterpret_cast<const uint8_t *>(&s_codes[warp][0]);
                    const int64_t e_end = min(c0 + (int64_t)kChunkCodes, n);
                    const int64_t p_lo = (c0 + pix_c - 1) / pix_c;      // first pixel that starts in this chunk
                    const int64_t p_hi = e_end / pix_c;                 // one past the last pixel that ends in it
                    unsigned *x4 = reinterpret_cast<unsigned *>(xe);
                    int64_t p_first = p_lo, p_last = p_hi;       // pixels [p_first, p_last) go one by one below
                    if (pl.s2d) {
                        // Space-to-depth image: horizontally adjacent pixels (2q, 2q + 1) are 2c contiguous bytes of one
                        // 16-byte block, so whole pairs go out as one or two aligned stores; the (at most two) single
                        // pixels at the chunk's ends take the pixel-by-pixel route.  Pixel counts fit 32 bits (host check).
                        const unsigned q_lo = (unsigned)((p_lo + 1) >> 1), q_hi = (unsigned)(p_hi >> 1);
                        const unsigned hw = (unsigned)(pl.H * pl.W), half_w = (unsigned)(pl.W >> 1);
                        // image coordinates of this lane's first pair by division, of its later pairs (64 pixels
                        // further on each) by stepping; the pair's bytes come out of shared memory as three aligned
                        // words and two funnel shifts
                        unsigned img = 0, h = 0, w = 0;
                        {
                            const unsigned px0 = 2u * (q_lo + lane);
                            img = px0 / hw;
                            const unsigned rem = px0 - img * hw;
                            h = rem / (unsigned)pl.W;
                            w = rem - h * (unsigned)pl.W;
                        }
                        const unsigned *sw32 = reinterpret_cast<const unsigned *>(sb);
                        int o0 = (int)((int64_t)(2u * (q_lo + lane)) * pix_c - c0);
                        for (unsigned q = q_lo + lane; q < q_hi; q += 32, o0 += 64 * pix_c, w += 64) {
                            while (w >= (unsigned)pl.W) {
                                w -= (unsigned)pl.W;
                                if (++h == (unsigned)pl.H) {
                                    h = 0;
                                    ++img;
                                }
                            }
                            uint8_t *row = xe + (((int64_t)(img * (unsigned)pl.Hs + (h >> 1)) * pl.P) << 4);
                            uint8_t *blk = row + (((w >> 1) + pl.padL) << 4);
                            const int wi = o0 >> 2;
                            const unsigned sh = (unsigned)(o0 & 3) * 8u;
                            const unsigned w0 = sw32[wi], w1 = sw32[min(wi + 1, kChunkCodes / 4 - 1)],
                                           w2 = sw32[min(wi + 2, kChunkCodes / 4 - 1)];
                            const unsigned long long v = (unsigned long long)__funnelshift_r(w0, w1, sh) |
                                                         ((unsigned long long)__funnelshift_r(w1, w2, sh) << 32);
                            const unsigned dy = h & 1u;
                            uint8_t *dst = blk + dy * 2 * pix_c;
                            if (pix_c == 3) {
                                if (dy == 0) {
                                    *reinterpret_cast<unsigned *>(dst) = (unsigned)v;
                                    *reinterpret_cast<unsigned short *>(dst + 4) = (unsigned short)(v >> 32);
                                } else {
                                    *reinterpret_cast<unsigned short *>(dst) = (unsigned short)v;
                                    *reinterpret_cast<unsigned *>(dst + 2) = (unsigned)(v >> 16);
                                    *reinterpret_cast<unsigned *>(blk + 12) = 0u;
                                }
                            } else if (pix_c == 4) {
                                *reinterpret_cast<uint2 *>(dst) = make_uint2((unsigned)v, (unsigned)(v >> 32));
                            } else if (pix_c == 2) {
                                *reinterpret_cast<unsigned *>(dst) = (unsigned)v;
                                if (dy) *reinterpret_cast<uint2 *>(blk + 8) = make_uint2(0u, 0u);
                            } else {
                                *reinterpret_cast<unsigned short *>(dst) = (unsigned short)v;
                                if (dy) {
                                    *reinterpret_cast<unsigned *>(blk + 4) = 0u;
                                    *reinterpret_cast<uint2 *>(blk + 8) = make_uint2(0u, 0u);
                                }
                            }
                            if (dy == 0) {
                                if (w == 0)
                                    for (int i = 0; i < pl.padL; ++i) reinterpret_cast<uint4 *>(row)[i] = make_uint4(0, 0, 0, 0);
                                if (w + 2 == (unsigned)pl.W)
                                    for (int i = 0; i < 3; ++i) reinterpret_cast<uint4 *>(row)[pl.padL + half_w + i] = make_uint4(0, 0, 0, 0);
                            }
                        }
                        // the single pixels: an odd first pixel and / or an even last one
                        p_first = p_hi;
                        p_last = p_hi;
                        if (lane == 2 && (p_lo & 1) && p_lo < p_hi) { p_first = p_lo; p_last = p_lo + 1; }
                        if (lane == 3 && (p_hi & 1) && p_hi - 1 >= p_lo) { p_first = p_hi - 1; p_last = p_hi; }
                    }
                    for (int64_t px = p_first + (pl.s2d ? 0 : lane); px < p_last; px += 32) {
                        const int o0 = (int)(px * pix_c - c0);
                        unsigned w = sb[o0];
                        if (pix_c > 1) w |= (unsigned)sb[o0 + 1] << 8;
                        if (pix_c > 2) w |= (unsigned)sb[o0 + 2] << 16;
                        if (pix_c > 3) w |= (unsigned)sb[o0 + 3] << 24;
                        if (pl.s2d) s2d_store_pixel(xe, pl, px, w);
                        else x4[px] = w;
                    }
                    if (lane == 0 && p_lo * pix_c > c0 && c0 < e_end) {
                        // tail of the pixel that began in the previous chunk
                        const int64_t px = p_lo - 1;
                        if (pl.s2d) {
                            uint8_t *dst = s2d_pixel_addr(xe, pl, px);
                            for (int64_t e = c0; e < min(p_lo * pix_c, e_end); ++e) dst[e - px * pix_c] = sb[e - c0];
                            if (p_lo * pix_c <= e_end) s2d_pixel_duties(xe, pl, px);      // the pixel ends in this chunk
                        } else {
                            for (int64_t e = c0; e < min(p_lo * pix_c, e_end); ++e) xe[px * 4 + (e - px * pix_c)] = sb[e - c0];
                        }
                    }
                    if (lane == 1 && p_hi * pix_c < e_end && p_hi >= p_lo) {
                        // head of the pixel that ends in the next chunk, and its padding bytes
                        const int64_t px = p_hi;
                        if (pl.s2d) {
                            uint8_t *dst = s2d_pixel_addr(xe, pl, px);
                            for (int64_t e = px * pix_c; e < e_end; ++e) dst[e - px * pix_c] = sb[e - c0];
                        } else {
                            for (int64_t e = px * pix_c; e < e_end; ++e) xe[px * 4 + (e - px * pix_c)] = sb[e - c0];
                            for (int b = pix_c; b < 4; ++b) xe[px * 4 + b] = 0;
                        }
                    }
                } else {
                if (off + 16 <= xe_bytes) reinterpret_cast<uint4 *>(xe + off)[0] = make_uint4(o[0], o[1], o[2], o[3]);
                if (off + 32 <= xe_bytes) reinterpret_cast<uint4 *>(xe + off)[1] = make_uint4(o[4], o[5], o[6], o[7]);
                }
            } else {
                unsigned o[16];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    o[2 * i] = (unsigned)s_lut[cw[i] & 0xffu] | ((unsigned)s_lut[(cw[i] >> 8) & 0xffu] << 16);
                    o[2 * i + 1] = (unsigned)s_lut[(cw[i] >> 16) & 0xffu] | ((unsigned)s_lut[cw[i] >> 24] << 16);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (off + 16 * (i + 1) <= xe_bytes)
                        reinterpret_cast<uint4 *>(xe + off)[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
            }
        }
        unsigned w[BITS];
        pack32<BITS>(cw, w);
        uint8_t *dst = packed + item * kChunkBytes;
        if (!DYBIT_CHECK(item * kChunkBytes + (int64_t)nvec * 16 <= packed_bytes, 0x24)) continue;
        if constexpr (BITS == 4) {
            if (lane < nvec) reinterpret_cast<uint4 *>(dst)[lane] = make_uint4(w[0], w[1], w[2], w[3]);
        } else if constexpr (BITS == 8) {
            if (2 * lane < nvec) reinterpret_cast<uint4 *>(dst)[2 * lane] = make_uint4(w[0], w[1], w[2], w[3]);
            if (2 * lane + 1 < nvec) reinterpret_cast<uint4 *>(dst)[2 * lane + 1] = make_uint4(w[4], w[5], w[6], w[7]);
        } else if constexpr (BITS == 2) {
            if ((lane >> 1) < nvec) reinterpret_cast<uint2 *>(dst)[lane] = make_uint2(w[0], w[1]);
        } else {
#pragma unroll
            for (int i = 0; i < BITS; ++i) s_words[warp][lane * BITS + i] = w[i];
            __syncwarp();
            const uint4 *s4 = reinterpret_cast<const uint4 *>(&s_words[warp][0]);
            for (int i = lane; i < nvec; i += 32) reinterpret_cast<uint4 *>(dst)[i] = s4[i];
        }
        __syncwarp();
    }
}

template <int BITS, bool SIGNED, int ELEM>
__global__ void __launch_bounds__(kStreamThreads, 3)
quantize_expand_kernel(const __grid_constant__ QeArgs a, const __grid_constant__ ElemTable tx, const __grid_constant__ ElemTable tw,
                       const __grid_constant__ XTab4 xt) {
    quantize_expand_body<BITS, SIGNED, ELEM>(a, tx, tw, xt, (int)blockIdx.x, (int)gridDim.x);
}

// The same for several layers of equal formats in ONE launch: blocks [first_block[l], first_block[l + 1]) work on
// layer l.
struct QeLayers {
    int n_layers;
    int first_block[kMaxGroupLayers + 1];
    QeArgs L[kMaxGroupLayers];
};

template <int BITS, bool SIGNED, int ELEM>
__global__ void __launch_bounds__(kStreamThreads, 3)
quantize_expand_layers_kernel(const __grid_constant__ QeLayers g, const __grid_constant__ ElemTable tx,
                              const __grid_constant__ ElemTable tw, const __grid_constant__ XTab4 xt) {
    int l = 0;
    while (l + 1 < g.n_layers && (int)blockIdx.x >= g.first_block[l + 1]) ++l;
    quantize_expand_body<BITS, SIGNED, ELEM>(g.L[l], tx, tw, xt, (int)blockIdx.x - g.first_block[l],
                                             g.first_block[l + 1] - g.first_block[l]);
}

// Arguments and grid share of one layer.  `one_wave`: the launch is this layer's alone, so its grid is what fits
// the GPU at once (three blocks per SM) and the activation's blocks loop over the chunks; otherwise (several layers
// in one launch, many waves) a warp takes about four chunks.
static QeArgs make_qe_args(const float *x, int64_t n, dybit_fmt fx, int elem, const float *scale, uint8_t *packed,
                           int64_t packed_bytes, uint8_t *xe, int64_t xe_bytes, const FusedWeights &wj,
                           const unsigned *partials, int n_partials, float *scale_out, const PixLayout &pl, bool one_wave,
                           int *blocks) {
    const int64_t chunk_bytes = (int64_t)kChunkCodes * fx.bits / 8;
    const int64_t resident = (int64_t)sm_count() * 3;
    const int64_t w_chunks = wj.pix_c > 0 ? wj.rows * (wj.out_stride / 16) : wj.rows * (wj.cols * elem / 16);
    int64_t w_blocks = (w_chunks + kStreamThreads * 4 - 1) / (kStreamThreads * 4);
    if (w_blocks > sm_count()) w_blocks = sm_count();
    if (w_blocks < 1) w_blocks = 1;
    const int64_t chunks = (packed_bytes + chunk_bytes - 1) / chunk_bytes;
    int64_t x_blocks = (chunks + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (one_wave) {
        if (x_blocks > resident - w_blocks) x_blocks = resident - w_blocks;
    } else {
        // (the pixel-by-pixel layouts of few-channel images are a long chain per chunk: one chunk per warp there)
        const int cpw = pl.c > 0 ? 1 : 4;
        x_blocks = (x_blocks + cpw - 1) / cpw;
        if (x_blocks > (1 << 20)) x_blocks = 1 << 20;
    }
    if (x_blocks < 1) x_blocks = 1;
    QeArgs a = {};
    a.x = x;
    a.n = n;
    a.scale = scale;
    a.packed = packed;
    a.packed_bytes = packed_bytes;
    a.xe = xe;
    a.xe_bytes = xe_bytes;
    a.wj = wj;
    a.x_blocks = (int)x_blocks;
    a.partials = partials;
    a.n_partials = n_partials;
    a.m = mag_bits(fx);
    a.scale_out = scale_out;
    a.pl = pl;
    *blocks = (int)(x_blocks + w_blocks);
    return a;
}

template <int BITS, bool SIGNED, int ELEM>
static dybit_status launch_qe_inst(const QeArgs &a, int blocks, const ElemTable &tx, const ElemTable &tw, const XTab4 &xt,
                                   cudaStream_t s) {
    launch_k(quantize_expand_kernel<BITS, SIGNED, ELEM>, dim3((unsigned)blocks), dim3((unsigned)kStreamThreads), (size_t)0, s, a, tx,
             tw, xt);
    return launch_status();
}

template <int BITS, bool SIGNED, int ELEM>
static dybit_status launch_qe_layers_inst(const QeLayers &g, int blocks, const ElemTable &tx, const ElemTable &tw,
                                          const XTab4 &xt, cudaStream_t s) {
    launch_k(quantize_expand_layers_kernel<BITS, SIGNED, ELEM>, dim3((unsigned)blocks), dim3((unsigned)kStreamThreads), (size_t)0, s,
             g, tx, tw, xt);
    return launch_status();
}

using QeLaunch = dybit_status (*)(const QeArgs &, int, const ElemTable &, const ElemTable &, const XTab4 &, cudaStream_t);
using QeLayersLaunch = dybit_status (*)(const QeLayers &, int, const ElemTable &, const ElemTable &, const XTab4 &, cudaStream_t);

template <int BITS, int ELEM>
static void qe_launchers_bits(bool sg, QeLaunch *one, QeLayersLaunch *many) {
    *one = sg ? launch_qe_inst<BITS, true, ELEM> : launch_qe_inst<BITS, false, ELEM>;
    *many = sg ? launch_qe_layers_inst<BITS, true, ELEM> : launch_qe_layers_inst<BITS, false, ELEM>;
}

template <int ELEM>
static bool qe_launchers(dybit_fmt fx, QeLaunch *one, QeLayersLaunch *many) {
    const bool sg = fx.is_signed != 0;
    switch (fx.bits) {
        case 2: qe_launchers_bits<2, ELEM>(sg, one, many); return true;
        case 3: qe_launchers_bits<3, ELEM>(sg, one, many); return true;
        case 4: qe_launchers_bits<4, ELEM>(sg, one, many); return true;
        case 5: qe_launchers_bits<5, ELEM>(sg, one, many); return true;
        case 6: qe_launchers_bits<6, ELEM>(sg, one, many); return true;
        case 7: qe_launchers_bits<7, ELEM>(sg, one, many); return true;
        case 8: qe_launchers_bits<8, ELEM>(sg, one, many); return true;
    }
    return false;
}

// Layers gathered for dybit_quantize_expand_layers: their max-abs reductions go out as one launch per
// kMaxGroupLayers tensors, their quantize + expand work as one launch per group of layers with equal formats.
struct QeGroupHost {
    dybit_fmt fx, fw;
    int elem;
    const ElemTable *tx, *tw;
    XTab4 xt;
    QeLayersLaunch launch;
    QeLayers g;
    int blocks;
};

struct LayerCollector {
    std::vector<AbsmaxLayers> absmax;
    std::vector<QeGroupHost> groups;

    dybit_status add_absmax(const float *x, int64_t n, unsigned *partials, int *n_partials) {
        int64_t blocks = (n / 4 + kStreamThreads * 16 - 1) / (kStreamThreads * 16);
        if (blocks > kMaxAbsmaxPartials) blocks = kMaxAbsmaxPartials;
        if (blocks < 1) blocks = 1;
        if (absmax.empty() || absmax.back().n_layers == kMaxGroupLayers) {
            absmax.emplace_back();
            absmax.back().n_layers = 0;
            absmax.back().first_block[0] = 0;
        }
        AbsmaxLayers &g = absmax.back();
        const int l = g.n_layers++;
        g.x[l] = x;
        g.n[l] = n;
        g.partials[l] = partials;
        g.first_block[l + 1] = g.first_block[l] + (int)blocks;
        *n_partials = (int)blocks;
        return DYBIT_OK;
    }

    dybit_status add_qe(dybit_fmt fx, dybit_fmt fw, int elem, const ElemTable &tx, const ElemTable &tw, const XTab4 &xt,
                        QeLayersLaunch launch, const QeArgs &a, int blocks) {
        QeGroupHost *grp = nullptr;
        for (QeGroupHost &c : groups)
            if (c.fx.bits == fx.bits && c.fx.is_signed == fx.is_signed && c.fw.bits == fw.bits && c.fw.is_signed == fw.is_signed &&
                c.elem == elem && c.tx == &tx && c.tw == &tw && c.g.n_layers < kMaxGroupLayers)
                grp = &c;
        if (grp == nullptr) {
            groups.emplace_back();
            grp = &groups.back();
            grp->fx = fx;
            grp->fw = fw;
            grp->elem = elem;
            grp->tx = &tx;
            grp->tw = &tw;
            grp->xt = xt;
            grp->launch = launch;
            grp->g.n_layers = 0;
            grp->g.first_block[0] = 0;
            grp->blocks = 0;
        }
        const int l = grp->g.n_layers++;
        grp->g.L[l] = a;
        grp->g.first_block[l + 1] = grp->g.first_block[l] + blocks;
        grp->blocks += blocks;
        return DYBIT_OK;
    }

    dybit_status launch_all(cudaStream_t s) {
        for (const AbsmaxLayers &g : absmax) {
            launch_k(absmax_layers_kernel, dim3((unsigned)g.first_block[g.n_layers]), dim3((unsigned)kStreamThreads), (size_t)0, s, g);
            if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
        }
        for (const QeGroupHost &c : groups) {
            const dybit_status st = c.launch(c.g, c.blocks, *c.tx, *c.tw, c.xt, s);
            if (st != DYBIT_OK) return st;
        }
        return DYBIT_OK;
    }
};

// One operand's expand job: rows of `cols` codes -> rows of container elements.
struct ExpandOperand {
    const uint8_t *packed;
    int bits;
    int64_t rows, in_stride, cols;
    uint8_t *out;
    int64_t out_stride;
    const ElemTable *table;
};

// True when the 4-bit register-table kernel applies: 1-byte container, whole 32-code vectors, and a table
// whose low half is non-negative and whose high half is either non-negative or the negated low-half style.
static bool expand4_job(const ExpandOperand &op, int elem, bool int8_container, Expand4Job *job) {
    if (op.bits != 4 || elem != 1 || op.cols % 32 != 0 || op.rows <= 0) return false;
    if (op.rows > 1 && (op.in_stride % 16 != 0 || op.out_stride % 16 != 0)) return false;
    int8_t v[16];
    for (int c = 0; c < 16; ++c) v[c] = (int8_t)(op.table->v[c] & 0xff);
    bool low_ok = true, high_pos = true, high_neg = true;
    for (int c = 0; c < 8; ++c) low_ok = low_ok && v[c] >= 0;
    for (int c = 8; c < 16; ++c) {
        high_pos = high_pos && v[c] >= 0;
        high_neg = high_neg && int8_container && v[c] <= 0 && v[c] > -128;   // two's complement only
    }
    if (!low_ok || !(high_pos || high_neg)) return false;
    job->packed = op.packed;
    job->out = op.out;
    job->rows = op.rows;
    job->in_stride = op.in_stride;
    job->out_stride = op.out_stride;
    job->vecs_per_row = op.cols / 32;
    job->neg_high = high_pos ? 0 : 1;
    for (int w = 0; w < 4; ++w) {
        unsigned word = 0;
        for (int b = 0; b < 4; ++b) {
            const int c = w * 4 + b;
            const int mag = (c >= 8 && !high_pos) ? -v[c] : v[c];
            word |= (unsigned)(mag & 0xff) << (8 * b);
        }
        job->tab[w] = word;
    }
    return true;
}

// Patch matrix for convolutions with few channels (pixel = neither 64 nor a multiple of 128 container
// bytes, e.g. the 3-channel stem): row m = output pixel, columns = the R*S*C taps in (r, s, c) order,
// decoded straight from the packed activation stream, zero where a tap falls outside the image, rows
// padded with zeros to krow bytes.  One thread assembles one row in shared memory (for a fixed r the
// S*C codes of the window are contiguous in NHWC); the block then writes its rows out coalesced.
struct PatchParams {
    const uint8_t *packed;     // dense NHWC code stream
    int64_t packed_words;      // its length in 32-bit words
    uint8_t *out;              // [M][krow] container bytes
    int bits, elem;
    int H, W, C, R, S, OH, OW, stride, pad, dil;
    int M, krow, row_pitch;    // row_pitch = krow + 4: odd word count, so threads hit distinct banks
};

__global__ void __launch_bounds__(128)
patch_expand_kernel(const PatchParams p, const __grid_constant__ ElemTable table) {
    extern __shared__ __align__(16) uint8_t s_rows[];
    __shared__ uint16_t s_lut[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = table.v[i];
    // zero everything first: padding taps and the row tail stay zero
    for (int i = threadIdx.x; i < (128 * p.row_pitch) / 4; i += blockDim.x) reinterpret_cast<unsigned *>(s_rows)[i] = 0u;
    __syncthreads();
    pdl_enter();
    const int m = blockIdx.x * 128 + threadIdx.x;
    if (m < p.M) {
        const int img = m / (p.OH * p.OW);
        const int rem = m - img * (p.OH * p.OW);
        const int oh = rem / p.OW, ow = rem - oh * p.OW;
        const int ih0 = oh * p.stride - p.pad, iw0 = ow * p.stride - p.pad;
        const unsigned mask = (1u << p.bits) - 1u;
        uint8_t *row = s_rows + threadIdx.x * p.row_pitch;
        const unsigned *w32 = reinterpret_cast<const unsigned *>(p.packed);
        for (int fr = 0; fr < p.R; ++fr) {
            const int ih = ih0 + fr * p.dil;
            if ((unsigned)ih >= (unsigned)p.H) continue;
            if (p.dil == 1) {
                // the taps of one filter row that fall inside the image are one contiguous run of codes
                const int s_lo = max(0, -iw0), s_hi = min(p.S, p.W - iw0);
                if (s_lo >= s_hi) continue;
                const int64_t bit = ((((int64_t)img * p.H + ih) * p.W + (iw0 + s_lo)) * p.C) * p.bits;
                uint8_t *dst = row + ((fr * p.S + s_lo) * p.C) * p.elem;
                const int count = (s_hi - s_lo) * p.C;
                if ((32 % p.bits) == 0) {
                    // 2-, 4- and 8-bit codes never straddle a 32-bit word: peel them off word by word
                    const int per_word = 32 / p.bits;
                    const int log_pw = p.bits == 2 ? 4 : (p.bits == 4 ? 3 : 2);
                    int64_t ci = bit >> (5 - log_pw);                 // global code index = bit / bits
                    int left = count, c = 0;
                    while (left > 0) {
                        const int k0 = (int)(ci & (per_word - 1));
                        const int take = min(per_word - k0, left);
                        unsigned word = __ldg(w32 + (ci >> log_pw)) >> (k0 * p.bits);
                        for (int t = 0; t < take; ++t, ++c) {
                            const unsigned v = s_lut[word & mask];
                            word >>= p.bits;
                            if (p.elem == 1) dst[c] = (uint8_t)v;
                            else reinterpret_cast<uint16_t *>(dst)[c] = (uint16_t)v;
                        }
                        ci += take;
                        left -= take;
                    }
                    continue;
                }
                // other widths: 64-bit window over the stream, refilled one word at a time
                int64_t wi = bit >> 5;
                const int sh = (int)(bit & 31);
                unsigned long long buf = __ldg(w32 + wi);
                if (wi + 1 < p.packed_words) buf |= (unsigned long long)__ldg(w32 + wi + 1) << 32;
                buf >>= sh;
                int avail = 64 - sh;
                wi += 2;
                for (int c = 0; c < count; ++c) {
                    if (avail < p.bits) {
                        if (wi < p.packed_words) buf |= (unsigned long long)__ldg(w32 + wi) << avail;
                        ++wi;
                        avail += 32;
                    }
                    const unsigned v = s_lut[(unsigned)buf & mask];
                    buf >>= p.bits;
                    avail -= p.bits;
                    if (p.elem == 1) dst[c] = (uint8_t)v;
                    else reinterpret_cast<uint16_t *>(dst)[c] = (uint16_t)v;
                }
                continue;
            }
            for (int fs = 0; fs < p.S; ++fs) {
                const int iw = iw0 + fs * p.dil;
                if ((unsigned)iw >= (unsigned)p.W) continue;
                int64_t bit = ((((int64_t)img * p.H + ih) * p.W + iw) * p.C) * p.bits;
                uint8_t *dst = row + ((fr * p.S + fs) * p.C) * p.elem;
                for (int c = 0; c < p.C; ++c, bit += p.bits) {
                    const int sh = (int)(bit & 7);
                    unsigned two = __ldg(p.packed + (bit >> 3));
                    if (sh + p.bits > 8) two |= (unsigned)__ldg(p.packed + (bit >> 3) + 1) << 8;
                    const unsigned v = s_lut[(two >> sh) & mask];
                    if (p.elem == 1) dst[c] = (uint8_t)v;
                    else reinterpret_cast<uint16_t *>(dst)[c] = (uint16_t)v;
                }
            }
        }
    }
    __syncthreads();
    // rows [blockIdx*128, +128) x krow bytes, 16 bytes per thread per step
    const int vec_per_row = p.krow / 16;
    const int rows_here = min(128, p.M - blockIdx.x * 128);
    for (int i = threadIdx.x; i < rows_here * vec_per_row; i += blockDim.x) {
        const int r = i / vec_per_row, v = i - r * vec_per_row;
        const unsigned *src = reinterpret_cast<const unsigned *>(s_rows + r * p.row_pitch + v * 16);
        const uint4 val = make_uint4(src[0], src[1], src[2], src[3]);
        *reinterpret_cast<uint4 *>(p.out + ((int64_t)blockIdx.x * 128 + r) * p.krow + v * 16) = val;
    }
}

// The same patch matrix from the activation's container elements in dense NHWC order (one element per code,
// no channel padding), for dilation 1: the taps of one filter row that fall inside the image are one
// contiguous byte run there, copied with aligned 32-bit loads and a funnel shift; the row is assembled
// word by word through a 64-bit accumulator (no byte stores, no table lookups), zeros where taps fall outside.
// The source must be readable up to 7 bytes past its last element.
struct PatchGatherParams {
    const uint8_t *xd;         // dense NHWC container elements
    uint8_t *out;              // [M][krow] container bytes
    int elem;
    int H, W, C, R, S, OH, OW, stride, pad;
    int M, krow, row_pitch;    // row_pitch = krow + 4: odd word count, so threads hit distinct banks
};

__global__ void __launch_bounds__(128)
patch_gather_kernel(const PatchGatherParams p) {
    extern __shared__ __align__(16) uint8_t s_rows[];
    pdl_enter();
    const int m = blockIdx.x * 128 + threadIdx.x;
    if (m < p.M) {
        const int img = m / (p.OH * p.OW);
        const int rem = m - img * (p.OH * p.OW);
        const int oh = rem / p.OW, ow = rem - oh * p.OW;
        const int ih0 = oh * p.stride - p.pad, iw0 = ow * p.stride - p.pad;
        const int tapb = p.C * p.elem;             // bytes per tap
        const int rowb = p.S * tapb;               // bytes per filter row
        const int s_lo = max(0, -iw0), s_hi = min(p.S, p.W - iw0);
        unsigned *wp = reinterpret_cast<unsigned *>(s_rows + threadIdx.x * p.row_pitch);
        unsigned long long acc = 0;
        int nb = 0;                                // bytes waiting in acc (always < 4 between steps)
        int zeros = 0;                             // zero bytes owed before the next run
        for (int fr = 0; fr < p.R; ++fr) {
            const int ih = ih0 + fr;
            if ((unsigned)ih >= (unsigned)p.H || s_lo >= s_hi) {
                zeros += rowb;
                continue;
            }
            nb += zeros + s_lo * tapb;
            while (nb >= 4) {
                *wp++ = (unsigned)acc;
                acc >>= 32;
                nb -= 4;
            }
            const int len = (s_hi - s_lo) * tapb;
            const int64_t a = (((int64_t)img * p.H + ih) * p.W + (iw0 + s_lo)) * tapb;
            const unsigned *src = reinterpret_cast<const unsigned *>(p.xd + (a & ~(int64_t)3));
            const unsigned sh = (unsigned)(a & 3) * 8u;
            unsigned w0 = __ldg(src);
            for (int j = 0; j < len; j += 4) {
                const unsigned w1 = __ldg(++src);
                unsigned v = __funnelshift_r(w0, w1, sh);
                w0 = w1;
                const int k = min(4, len - j);
                if (k < 4) v &= (1u << (8 * k)) - 1u;
                acc |= (unsigned long long)v << (8 * nb);
                nb += k;
                if (nb >= 4) {
                    *wp++ = (unsigned)acc;
                    acc >>= 32;
                    nb -= 4;
                }
            }
            zeros = (p.S - s_hi) * tapb;
        }
        // zeros owed, then the row's zero tail up to krow (a multiple of 16, so nothing is left over)
        nb += zeros + p.krow - p.R * rowb;
        while (nb >= 4) {
            *wp++ = (unsigned)acc;
            acc >>= 32;
            nb -= 4;
        }
    }
    __syncthreads();
    const int vec_per_row = p.krow / 16;
    const int rows_here = min(128, p.M - blockIdx.x * 128);
    for (int i = threadIdx.x; i < rows_here * vec_per_row; i += blockDim.x) {
        const int r = i / vec_per_row, v = i - r * vec_per_row;
        const unsigned *src = reinterpret_cast<const unsigned *>(s_rows + r * p.row_pitch + v * 16);
        const uint4 val = make_uint4(src[0], src[1], src[2], src[3]);
        *reinterpret_cast<uint4 *>(p.out + ((int64_t)blockIdx.x * 128 + r) * p.krow + v * 16) = val;
    }
}

// Packed NHWC codes with C <= 4 channels -> one 32-bit word per pixel (C one-byte elements, zero padding), and the
// weights in the matching filter-row layout (expand_weights_pix4), in one launch: blocks [0, x_blocks) take pixels.
__global__ void __launch_bounds__(256)
expand_pix4_kernel(const uint8_t *__restrict__ packed, int bits, int64_t pixels, int c, unsigned *__restrict__ x4,
                   const __grid_constant__ ElemTable tx, const FusedWeights wj, const __grid_constant__ ElemTable tw,
                   int x_blocks, const PixLayout pl) {
    __shared__ uint16_t s_lut[256];
    const bool weights = (int)blockIdx.x >= x_blocks;
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = weights ? tw.v[i] : tx.v[i];
    __syncthreads();
    pdl_enter();
    if (weights) {
        const int64_t total = wj.rows * (wj.out_stride / 16);
        for (int64_t idx = (int64_t)(blockIdx.x - x_blocks) * blockDim.x + threadIdx.x; idx < total;
             idx += (int64_t)(gridDim.x - x_blocks) * blockDim.x) {
            if (wj.s2d) expand_weights_s2d(wj, s_lut, idx);
            else expand_weights_pix4(wj, s_lut, idx);
        }
        return;
    }
    const unsigned mask = (1u << bits) - 1u;
    for (int64_t px = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; px < pixels; px += (int64_t)x_blocks * blockDim.x) {
        unsigned w = 0;
        int64_t bit = px * c * bits;
        for (int ch = 0; ch < c; ++ch, bit += bits) {
            const int sh = (int)(bit & 7);
            unsigned two = __ldg(packed + (bit >> 3));
            if (sh + bits > 8) two |= (unsigned)__ldg(packed + (bit >> 3) + 1) << 8;
            w |= (unsigned)(s_lut[(two >> sh) & mask] & 0xffu) << (8 * ch);
        }
        if (pl.s2d) s2d_store_pixel(reinterpret_cast<uint8_t *>(x4), pl, px, w);
        else x4[px] = w;
    }
}

template <int ELEM>
static dybit_status launch_expand_rows(const uint8_t *packed, int bits, int64_t rows, int64_t in_stride, int64_t cols,
                                       uint8_t *out, int64_t out_stride, const ElemTable &t, cudaStream_t s) {
    // rows that follow one another without gaps on both sides are one flat run of codes: short rows (a K of 64 is
    // 128 codes) then fill whole 1024-code chunks instead of an eighth of one
    if (rows > 1 && in_stride * 8 == cols * bits && out_stride == cols * ELEM) {
        cols *= rows;
        rows = 1;
    }
    const int64_t items = rows * ((cols + kChunkCodes - 1) / kChunkCodes);
    if (items == 0) return DYBIT_OK;
    const int grid = stream_grid((items + 1) / 2);
    switch (bits) {
        case 2: launch_k(expand_rows_kernel<2, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        case 3: launch_k(expand_rows_kernel<3, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        case 4: launch_k(expand_rows_kernel<4, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        case 5: launch_k(expand_rows_kernel<5, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        case 6: launch_k(expand_rows_kernel<6, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        case 7: launch_k(expand_rows_kernel<7, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        case 8: launch_k(expand_rows_kernel<8, ELEM>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, rows, in_stride, cols, out, out_stride, t); break;
        default: return DYBIT_ERR_INVALID_ARG;
    }
    return launch_status();
}

static dybit_status launch_expand(const uint8_t *packed, int bits, int64_t rows, int64_t in_stride, int64_t cols,
                                  int elem, uint8_t *out, int64_t out_stride, const ElemTable &t, cudaStream_t s) {
    return elem == 1 ? launch_expand_rows<1>(packed, bits, rows, in_stride, cols, out, out_stride, t, s)
                     : launch_expand_rows<2>(packed, bits, rows, in_stride, cols, out, out_stride, t, s);
}

// Expands both operands of a GEMM: one launch when both take the 4-bit register-table kernel.
static dybit_status launch_expand_pair(const ExpandOperand &a, const ExpandOperand &b, int elem, bool int8_container,
                                       cudaStream_t s) {
    Expand4Job ja, jb;
    const bool fa = expand4_job(a, elem, int8_container, &ja), fb = expand4_job(b, elem, int8_container, &jb);
    if (fa || fb) {
        Expand4Job none = {};
        const Expand4Job &j0 = fa ? ja : jb;
        const Expand4Job &j1 = (fa && fb) ? jb : none;
        const int64_t vecs0 = j0.rows * j0.vecs_per_row;
        const int64_t total = vecs0 + j1.rows * j1.vecs_per_row;
        int64_t blocks = (total + 255) / 256, cap = (int64_t)sm_count() * 16;
        if (blocks > cap) blocks = cap;
        launch_k(expand4_kernel, dim3((unsigned)((int)blocks)), dim3((unsigned)(256)), (size_t)(0), s, j0, j1, vecs0);
        if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
    }
    if (!fa) {
        dybit_status st = launch_expand(a.packed, a.bits, a.rows, a.in_stride, a.cols, elem, a.out, a.out_stride, *a.table, s);
        if (st != DYBIT_OK) return st;
    }
    if (!fb) {
        dybit_status st = launch_expand(b.packed, b.bits, b.rows, b.in_stride, b.cols, elem, b.out, b.out_stride, *b.table, s);
        if (st != DYBIT_OK) return st;
    }
    return DYBIT_OK;
}

// ------------------------------------------------------------------ the tcgen05 GEMM

constexpr int kBM = 128;            // tile rows (UMMA M)
constexpr int kBKBytes = 128;       // one 128-byte swizzle row of K per pipeline stage (64 in the SWB = 64 variant)
constexpr int kUmmaKBytes = 32;     // K bytes consumed by one tcgen05.mma
constexpr int kStageBytesTotal = 192 * 1024;
constexpr int kEpilogueWarps = 8;     // two groups of four (one warp per TMEM lane quarter in each)
constexpr unsigned long long kWaitLimitNs = 4000000000ull;

struct GemmParams {
    int M, N;                 // output extent
    int k_blocks;             // 128-byte K blocks per row
    int m_tiles, n_tiles;
    float *C;
    int32_t *C_raw;
    int64_t ldc;
    const float *scale_a, *scale_b;
    double pow2;              // alpha = (float)(scale_a * scale_b * pow2)
    // implicit-GEMM addressing of A (convolution only)
    const uint8_t *xe;        // expanded activation, [n*h*w][cpb] bytes
    int H, W, OH, OW, R, S, stride, pad, dil;
    int cpb;                  // bytes per pixel in xe (padded channels * element size)
    int kb_per_tap;           // im2col mode: SWB-byte blocks per filter tap (cpb / SWB)
    int b_resident;           // 1: one tile column and k_blocks <= stages: the whole B panel is loaded once per CTA
                              //    into the B stage slots (slot = K block) and the ring carries A only
    int tma_store;            // 1: C leaves through shared memory and TMA stores (needs 16-byte aligned C rows)
    // re-quantizing epilogue: when Q is set the result is encoded and packed instead of stored as fp32
    uint8_t *Q;               // row m starts at Q + m * ldq; N codes of q_bits each
    int64_t ldq;
    const float *scale_q;     // {scale, 1/scale} of the output tensor
    int q_bits, q_signed, relu;
    const float *bias;        // requant only: one fp32 per output column, or null
    unsigned long long *clock; // profiling: {min start after the dependency wait, max end} in %globaltimer ns, or null
    int bmt;                  // batched GEMM: M tiles per batch entry (0: not batched); M is then one entry's rows
    int split_from;           // pair kernel: tiles from this index on are worked on as two 256 x 128 halves (see pair_item)
    int64_t c_bstride;        // batched GEMM: elements between consecutive entries of C / C_raw
};

// Waits for the phase with the given parity; gives up after `limit_ns` (kWaitLimitNs in every kernel of the
// library), records the site in the device status word and raises the CTA-wide abort flag.
__device__ __forceinline__ bool wait_bounded(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                             unsigned site, unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    unsigned spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                atomicOr(&g_device_status, (site << 8) | 1u);
                *abort_flag = 1u;
                return false;
            }
        }
    }
}

// The same wait for the MMA-issuing thread: the barrier is named by its shared-memory address and only the first
// probe is inlined, so the common case (the stage is there already) costs three instructions.
__device__ __noinline__ bool wait_bounded_slow(uint32_t bar_addr, uint32_t parity, volatile uint32_t *abort_flag, unsigned site) {
    const uint64_t t0 = global_timer_ns();
    unsigned spins = 0;
    for (;;) {
        if (mbar_try_wait_addr(bar_addr, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                atomicOr(&g_device_status, (site << 8) | 1u);
                *abort_flag = 1u;
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool wait_bounded_addr(uint32_t bar_addr, uint32_t parity, volatile uint32_t *abort_flag,
                                                  unsigned site) {
    if (mbar_try_wait_addr(bar_addr, parity)) return true;
    return wait_bounded_slow(bar_addr, parity, abort_flag, site);
}

// Self-test of the give-up path: one thread waits, with the library's own wait_bounded, on a barrier that nothing
// ever arrives on.  The wait runs out after limit_ns, sets the status word (site kSelftestSite) and the abort flag
// and returns; result[0] receives 1 if the wait reported failure, result[1] the abort flag.
constexpr unsigned kSelftestSite = 0x5e;
__global__ void wait_timeout_selftest_kernel(unsigned long long limit_ns, unsigned *result) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_word;
    pdl_enter();
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_word = 0;
        fence_mbar_init();
        const bool got = wait_bounded(&bar, 0u, &abort_word, kSelftestSite, limit_ns);
        result[0] = got ? 0u : 1u;
        result[1] = abort_word;
    }
}

// How the A tile reaches shared memory.
enum AMode { kATiled = 0,    // GEMM: 2-D tiled TMA
             kAGather = 1,   // conv: four warps gather 16-byte chunks with cp.async (any channel count)
             kAIm2col = 2,   // conv: one im2col TMA per stage (pixel = a whole number of SWB-byte blocks)
             kAGather4 = 3 };// conv with <= 4 one-byte channels: pixels are 32-bit words, a K block = four filter rows of
                             // eight taps, gathered with 4-byte cp.async

// Re-quantizing epilogue (Section III-B.1: results are quantized to DyBit before they are written back):
// 32 consecutive outputs of one row -> 32 codes of the output format -> 4*BITS bytes at dst.
// `valid` < 32 only in the last column chunk; then only whole bytes of valid codes are written.
template <int BITS, bool SIGNED>
__device__ __noinline__ void requant_store32(const float *f, float inv, uint8_t *dst, int valid) {
    unsigned cw[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
        cw[j] = encode4<BITS, SIGNED>(make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]), inv);
    unsigned w[BITS];
    pack32<BITS>(cw, w);
    if (valid >= 32 && (reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
#pragma unroll
        for (int i = 0; i < BITS; ++i) reinterpret_cast<unsigned *>(dst)[i] = w[i];
    } else {
        const int bytes = (valid < 32 ? valid : 32) * BITS / 8;
        for (int b = 0; b < bytes; ++b) dst[b] = (uint8_t)(w[b >> 2] >> ((b & 3) * 8));
    }
}

// The same, fully inlined and fed from registers: used for the output widths the search space of
// Section III-C.3 selects (2, 4 and 8 bits); the other widths go through the out-of-line version.
template <int BITS, bool SIGNED>
__device__ __forceinline__ void requant_store32_inline(const float (&f)[32], float inv, uint8_t *dst, int valid) {
    unsigned cw[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
        cw[j] = encode4<BITS, SIGNED>(make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]), inv);
    unsigned w[BITS];
    pack32<BITS>(cw, w);
    if (valid >= 32 && (reinterpret_cast<uintptr_t>(dst) & (BITS == 2 ? 7 : 15)) == 0) {
        if constexpr (BITS == 2) *reinterpret_cast<uint2 *>(dst) = make_uint2(w[0], w[1]);
        else if constexpr (BITS == 4) *reinterpret_cast<uint4 *>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        else {
            reinterpret_cast<uint4 *>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
            reinterpret_cast<uint4 *>(dst)[1] = make_uint4(w[4 % BITS], w[5 % BITS], w[6 % BITS], w[7 % BITS]);
        }
    } else {
        const int bytes = (valid < 32 ? valid : 32) * BITS / 8;
        for (int b = 0; b < bytes; ++b) dst[b] = (uint8_t)(w[b >> 2] >> ((b & 3) * 8));
    }
}

__device__ __forceinline__ void requant_dispatch(int bits, int is_signed, const float (&f)[32], float inv, uint8_t *dst,
                                                 int valid) {
    switch (bits * 2 + is_signed) {
        case 4: requant_store32_inline<2, false>(f, inv, dst, valid); return;
        case 5: requant_store32_inline<2, true>(f, inv, dst, valid); return;
        case 8: requant_store32_inline<4, false>(f, inv, dst, valid); return;
        case 9: requant_store32_inline<4, true>(f, inv, dst, valid); return;
        case 16: requant_store32_inline<8, false>(f, inv, dst, valid); return;
        case 17: requant_store32_inline<8, true>(f, inv, dst, valid); return;
        default: break;
    }
    // the other widths run out of line on a copy, so that f itself can stay in registers
    float tmp[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) tmp[j] = f[j];
    switch (bits * 2 + is_signed) {
        case 6: requant_store32<3, false>(tmp, inv, dst, valid); break;
        case 7: requant_store32<3, true>(tmp, inv, dst, valid); break;
        case 10: requant_store32<5, false>(tmp, inv, dst, valid); break;
        case 11: requant_store32<5, true>(tmp, inv, dst, valid); break;
        case 12: requant_store32<6, false>(tmp, inv, dst, valid); break;
        case 13: requant_store32<6, true>(tmp, inv, dst, valid); break;
        case 14: requant_store32<7, false>(tmp, inv, dst, valid); break;
        case 15: requant_store32<7, true>(tmp, inv, dst, valid); break;
        default: break;
    }
}

template <int BN, int SWB>
struct GemmSmem {
    static constexpr int kAStage = kBM * SWB;
    static constexpr int kBStage = BN * SWB;
    static constexpr int kFit = kStageBytesTotal / (kAStage + kBStage);
    static constexpr int kStages = kFit > 12 ? 12 : kFit;
    static constexpr int kBarrierBytes = 512;
    static constexpr int kCStage = kBM * 128;                  // 128 rows x 32 fp32 columns of the output tile
    static constexpr int kBytes = kStages * (kAStage + kBStage) + 2 * kCStage + kBarrierBytes + 1024;   // + alignment slack
};

__device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, int &m_blk, int &n_blk) {
    // groups of 8 tile-rows sweep all tile-columns, so one wave of CTAs shares few A and B tiles
    constexpr int kGroup = 8;
    const int per_group = kGroup * n_tiles;
    const int group = tile / per_group;
    const int first_m = group * kGroup;
    const int gsz = min(kGroup, m_tiles - first_m);
    const int in_group = tile - group * per_group;
    m_blk = first_m + in_group % gsz;
    n_blk = in_group / gsz;
}

// CTA `bid` of the `nblk` CTAs that work on the problem (tensor maps and parameters live in the kernel's
// parameter space, whichever kernel below passes them).
template <Kind KIND, int BN, int AMODE, int SWB>
__device__ __forceinline__ void gemm_body(const CUtensorMap &tmap_a, const CUtensorMap &tmap_b, const CUtensorMap &tmap_c,
                                          const GemmParams &p, const int bid, const int nblk) {
    static_assert((AMODE != kAGather && AMODE != kAGather4) || SWB == 128, "the cp.async gather writes 128-byte rows");
    constexpr bool CONV = AMODE == kAGather || AMODE == kAGather4;          // extra gather warps present
    using L = GemmSmem<BN, SWB>;
    constexpr int kStages = L::kStages;
    constexpr int kGatherThreads = AMODE == kAGather4 ? 256 : 128;     // pixel-word mode: two threads per tile row
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_stages = smem;
    uint8_t *b_stages = smem + kStages * L::kAStage;
    uint8_t *c_stages = smem + kStages * (L::kAStage + L::kBStage);       // two output staging buffers
    uint64_t *bars = reinterpret_cast<uint64_t *>(c_stages + 2 * L::kCStage);
    uint64_t *full = bars;
    uint64_t *empty = bars + kStages;
    uint64_t *acc_full = bars + 2 * kStages;
    uint64_t *acc_empty = acc_full + 2;
    uint64_t *b_full = acc_empty + 2;                    // resident-B mode: the panel has landed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(b_full + 1);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = p.m_tiles * p.n_tiles;
    constexpr uint32_t kTmemCols = 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], CONV ? 1 + (AMODE == kAGather4 ? kGatherThreads / 32 : kGatherThreads) : 1);
            mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], kEpilogueWarps);
        }
        mbar_init(b_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
        if (!CONV) prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (p.tma_store) prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // The producer's coordinates of its first tile (a few integer divisions, ~0.7 us in a single thread) are worked
    // out before the wait below, so they overlap the predecessor's tail.  im2col mode: window origin of the
    // tile's first output pixel.
    struct TileOrigin { int m_blk, n_blk, iw, ih, img; };
    auto tile_origin = [&](int tile) {
        TileOrigin o = {0, 0, 0, 0, 0};
        tile_coords(tile, p.m_tiles, p.n_tiles, o.m_blk, o.n_blk);
        if (AMODE == kAIm2col) {
            const int m0 = o.m_blk * kBM;
            o.img = m0 / (p.OH * p.OW);
            const int rem = m0 - o.img * (p.OH * p.OW);
            const int oh = rem / p.OW;
            o.ih = oh * p.stride - p.pad;
            o.iw = (rem - oh * p.OW) * p.stride - p.pad;
        }
        return o;
    };
    TileOrigin first = {0, 0, 0, 0, 0};
    if (threadIdx.x == 0 && bid < total_tiles) {
        first = tile_origin(bid);
        asm volatile("" : "+r"(first.m_blk), "+r"(first.n_blk), "+r"(first.iw), "+r"(first.ih), "+r"(first.img));
    }
    // everything above touched only this CTA's own resources; operands, scales and outputs come next
    pdl_enter();
    if (p.clock != nullptr && threadIdx.x == 32) atomicMin(p.clock, (unsigned long long)global_timer_ns());

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const bool b_res = !CONV && p.b_resident != 0;
            if (b_res && bid < total_tiles) {
                // every tile of this CTA multiplies by the same B panel: fetch it once, K block kb into slot kb
                mbar_arrive_expect_tx(b_full, (uint32_t)p.k_blocks * L::kBStage);
                for (int kb = 0; kb < p.k_blocks; ++kb)
                    tma_load_2d(b_stages + kb * L::kBStage, &tmap_b, kb * SWB, 0, b_full);
            }
            for (int tile = bid; tile < total_tiles && ok; tile += nblk) {
                const TileOrigin o = tile == bid ? first : tile_origin(tile);
                const int m_blk = o.m_blk, n_blk = o.n_blk, iw = o.iw, ih = o.ih, img = o.img;
                int fr = 0, fs = 0, cb = 0;                     // im2col mode: the running filter tap
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!wait_bounded(&empty[s], ph ^ 1u, abort_flag, 1)) { ok = false; break; }
                    mbar_arrive_expect_tx(&full[s], CONV ? L::kBStage : (b_res ? L::kAStage : L::kAStage + L::kBStage));
                    if (AMODE == kATiled) {
                        if (p.bmt) tma_load_3d(a_stages + s * L::kAStage, &tmap_a, kb * SWB, (m_blk % p.bmt) * kBM, m_blk / p.bmt, &full[s]);
                        else tma_load_2d(a_stages + s * L::kAStage, &tmap_a, kb * SWB, m_blk * kBM, &full[s]);
                    } else if (AMODE == kAIm2col) {
                        tma_load_im2col_4d(a_stages + s * L::kAStage, &tmap_a, cb * SWB, iw, ih, img, &full[s],
                                           (uint16_t)(fs * p.dil), (uint16_t)(fr * p.dil));
                        if (++cb == p.kb_per_tap) {
                            cb = 0;
                            if (++fs == p.S) { fs = 0; ++fr; }
                        }
                    }
                    if (b_res) continue;
                    if (AMODE == kATiled && p.bmt) tma_load_3d(b_stages + s * L::kBStage, &tmap_b, kb * SWB, n_blk * BN, m_blk / p.bmt, &full[s]);
                    else tma_load_2d(b_stages + s * L::kBStage, &tmap_b, kb * SWB, n_blk * BN, &full[s]);
                }
            }
            if (!ok) {
                // give copies already in flight a bounded time to land before the CTA retires
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t kCFormat = (KIND == Kind::I8) ? 2u : 1u;           // s32 : f32
            constexpr uint32_t kABFormat = (KIND == Kind::F8F6F4) ? 0u : 1u;      // e4m3 : (s8 | bf16)
            constexpr uint32_t idesc = umma_idesc(kCFormat, kABFormat, kBM, BN);
            // One thread runs at roughly six clocks per instruction and an MMA of a narrow tile takes under 100, so
            // the loop is kept to 32-bit adds (descriptors = constant high word + stepped low word, barriers by
            // shared-memory address).  A barrier probed right after a tcgen05.commit answers only once the MMAs in
            // flight have drained (about 200 clocks; about 45 between two MMAs): the NEXT stage's barrier is probed
            // right after the first MMA of the current stage.  A wait that runs out raises the abort flag and the
            // loop simply runs on (later waits then give up at once; the epilogue stores nothing more).
            constexpr uint32_t kHi = umma_desc_hi<SWB>();
            constexpr uint32_t kA16 = L::kAStage >> 4, kB16 = L::kBStage >> 4;
            const uint32_t a_lo0 = umma_desc_lo(smem_u32(a_stages)), b_lo0 = umma_desc_lo(smem_u32(b_stages));
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty);
            const uint32_t acc_full0 = smem_u32(acc_full), acc_empty0 = smem_u32(acc_empty);
            const bool b_res = !CONV && p.b_resident != 0;
            const int k_blocks = p.k_blocks;
            int s = 0;
            uint32_t ph = 0, lt = 0;
            bool ready = false, acc_ready = false;
            if (b_res && bid < total_tiles) (void)wait_bounded(b_full, 0u, abort_flag, 6);
            for (int tile = bid; tile < total_tiles; tile += nblk, ++lt) {
                const uint32_t as = lt & 1u;
                if (!acc_ready) (void)wait_bounded_addr(acc_empty0 + as * 8, ((lt >> 1) & 1u) ^ 1u, abort_flag, 2);
                acc_ready = false;
                tc_fence_after_sync();
                const uint32_t d = tmem_base + as * BN;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!ready) (void)wait_bounded_addr(full0 + s * 8, ph, abort_flag, 3);
                    tc_fence_after_sync();
                    int sn = s + 1;
                    uint32_t phn = ph;
                    if (sn == kStages) { sn = 0; phn ^= 1u; }
                    const uint32_t a_lo = a_lo0 + s * kA16;
                    const uint32_t b_lo = b_lo0 + (b_res ? kb : s) * kB16;
                    umma_lo<KIND>(d, a_lo, b_lo, kHi, idesc, (uint32_t)(kb != 0));
                    ready = mbar_try_wait_addr(full0 + sn * 8, phn);
                    if (kb == k_blocks - 1)
                        acc_ready = mbar_try_wait_addr(acc_empty0 + (as ^ 1u) * 8, (((lt + 1) >> 1) & 1u) ^ 1u);
#pragma unroll
                    for (int k = 1; k < SWB / kUmmaKBytes; ++k)
                        umma_lo<KIND>(d, a_lo + k * (kUmmaKBytes >> 4), b_lo + k * (kUmmaKBytes >> 4), kHi, idesc, 1u);
                    umma_commit_addr(empty0 + s * 8);
                    s = sn;
                    ph = phn;
                }
                umma_commit_addr(acc_full0 + as * 8);
            }
        }
    } else if (warp < 2 + kEpilogueWarps) {
        // ------------------------------------------------ epilogue: TMEM -> registers -> (shared -> TMA store | global)
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int row_in_tile = q * 32 + lane;
        // two groups of four warps; group g takes the 32-column chunks cc = g, g + 2, ... and owns staging buffer g
        const int group = (warp - 2) >> 2;
        const bool issuer = (threadIdx.x & 127) == 64; // first lane of each group: issues and tracks its TMA stores
        const float alpha = (float)((double)__ldg(p.scale_a) * (double)__ldg(p.scale_b) * p.pow2);
        const float inv_q = p.Q ? __ldg(p.scale_q + 1) : 1.0f;
        const bool vec_ok = ((reinterpret_cast<uintptr_t>(p.C) & 15) == 0) && (p.ldc % 4 == 0) &&
                            (p.C_raw == nullptr || (reinterpret_cast<uintptr_t>(p.C_raw) & 15) == 0);
        uint32_t lt = 0;
        for (int tile = bid; tile < total_tiles; tile += nblk, ++lt) {
            int m_blk, n_blk;
            tile_coords(tile, p.m_tiles, p.n_tiles, m_blk, n_blk);
            const uint32_t as = lt & 1u, aph = (lt >> 1) & 1u;
            // The four warps of a group meet in named barriers below, so they must leave this loop together: the
            // outcome of the wait is AND-reduced over the group's 128 threads (every warp gets here in bounded time).
            // (one thread per group polls; the others sleep in the hardware barrier that hands them the outcome)
            const bool ok = named_barrier_and(1 + group, 128, issuer ? wait_bounded(&acc_full[as], aph, abort_flag, 4) : true);
            if (!ok) break;
            tc_fence_after_sync();
            // batched: the tile belongs to entry `bat`, rows count inside that entry
            const int bat = p.bmt ? m_blk / p.bmt : 0;
            const int m_loc = m_blk - bat * p.bmt;
            const int row = m_loc * kBM + row_in_tile;
            const uint32_t taddr = tmem_base + as * BN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int cc = group; cc < BN / 32; cc += kEpilogueWarps / 4) {
                const int col0 = n_blk * BN + cc * 32;
                if (col0 >= p.N) break;                // uniform over the group: the rest of the tile lies outside C
                uint32_t r[32];
                tmem_ld_32x32(taddr + cc * 32, r);
                tmem_ld_wait();
                float f[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float acc = (KIND == Kind::I8) ? __int2float_rn((int)r[j]) : __uint_as_float(r[j]);
                    f[j] = __fmul_rn(acc, alpha);
                }
                if (p.Q) {
                    if (row < p.M) {
                        if (p.bias) {
                            // every lane reads the same 32 floats: one broadcast transaction each
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < p.N) f[j] = __fadd_rn(f[j], __ldg(p.bias + col0 + j));
                        }
                        if (p.relu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.0f);
                        }
                        if (DYBIT_CHECK((int64_t)col0 * p.q_bits / 8 + (int64_t)min(32, p.N - col0) * p.q_bits / 8 <= p.ldq, 0x25))
                            requant_dispatch(p.q_bits, p.q_signed, f, inv_q,
                                             p.Q + (int64_t)row * p.ldq + (int64_t)col0 * p.q_bits / 8, p.N - col0);
                    }
                    continue;
                }
                if (p.tma_store) {
                    // stage 128 rows x 128 bytes in the TMA's 128-byte swizzle, then one thread stores the box;
                    // rows / columns beyond C are clipped by the tensor map.  In the CTA's last tile the operand
                    // stages are idle (the commit that published this accumulator followed the last MMA), so every
                    // chunk takes a buffer of its own there and no store waits for the one before it.
                    const bool last_tile = tile + nblk >= total_tiles;
                    uint8_t *stage = last_tile ? a_stages + cc * L::kCStage : c_stages + group * L::kCStage;
                    if (issuer && !last_tile) bulk_wait_group_read<0>();   // the store that last read this buffer is done with it
                    named_barrier(1 + group, 128);
                    uint8_t *srow = stage + row_in_tile * 128;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4 *>(srow + ((j ^ (row_in_tile & 7)) << 4)) =
                            make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                    fence_proxy_async_smem();
                    named_barrier(1 + group, 128);
                    if (issuer) {
                        if (p.bmt) tma_store_3d(&tmap_c, stage, col0, m_loc * kBM, bat);
                        else tma_store_2d(&tmap_c, stage, col0, m_blk * kBM);
                        bulk_commit_group();
                    }
                }
                if (!p.tma_store) {
                    // C cannot be described to the TMA (rows or base not 16-byte aligned): each warp stages its own
                    // 32 rows in the same buffer and writes them out row by row, 32 consecutive floats per store
                    uint8_t *stage = c_stages + group * L::kCStage;
                    __syncwarp();
                    uint8_t *srow = stage + row_in_tile * 128;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4 *>(srow + ((j ^ (row_in_tile & 7)) << 4)) =
                            make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                    __syncwarp();
                    const int col = col0 + lane;
                    const int r_first = m_loc * kBM + q * 32;
                    if (col < p.N) {
                        float *cout = p.C + (int64_t)bat * p.c_bstride + (int64_t)r_first * p.ldc + col;
                        const int rows_here = min(32, p.M - r_first);
                        for (int rr = 0; rr < rows_here; ++rr) {
                            const int rt = q * 32 + rr;
                            const float v = *reinterpret_cast<const float *>(stage + rt * 128 + (((lane >> 2) ^ (rt & 7)) << 4) + ((lane & 3) << 2));
                            __stcs(cout + (int64_t)rr * p.ldc, v);
                        }
                    }
                }
                if (row < p.M) {
                    const int64_t coff = (int64_t)bat * p.c_bstride + (int64_t)row * p.ldc + col0;
                    int32_t *rrow = p.C_raw ? p.C_raw + coff : nullptr;
                    if (vec_ok && col0 + 32 <= p.N) {
                        if (KIND == Kind::I8 && rrow) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                __stcs(reinterpret_cast<int4 *>(rrow) + j, make_int4((int)r[4 * j], (int)r[4 * j + 1], (int)r[4 * j + 2], (int)r[4 * j + 3]));
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (col0 + j < p.N) {
                                if (KIND == Kind::I8 && rrow) rrow[j] = (int)r[j];
                            }
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[as]);
        }
        if (issuer) bulk_wait_group_read<0>();             // shared memory must outlive the last store's read
    } else if (CONV) {
        // ------------------------------------------------ im2col gather of the A tile (4 warps, one row per thread)
        const int t = (threadIdx.x - 32 * (2 + kEpilogueWarps)) & 127;   // tile row 0..127
        const int half = (threadIdx.x - 32 * (2 + kEpilogueWarps)) >> 7;   // pixel-word mode: which two of a K block's four filter rows
        const int sw = t & 7;
        constexpr int kAhead = 2;                     // stages issued but not yet published
        uint32_t it = 0, issued = 0, published = 0;
        bool ok = true;
        if (AMODE == kAGather4) {
            // Pixel-word mode.  A K block of the A tile = four filter rows (4*kb ..) of eight 4-byte slots, slot s =
            // tap s; this thread fills two of the four rows of its tile row: plain loads (the pixel words are reused
            // by many windows and sit in L1) into registers, zeros where the tap does not exist or lies outside the
            // image, then one 16-byte shared-memory store per chunk.  The loads of the NEXT K block (possibly of the
            // next tile) are issued before this one's stage is waited for, so their latency hides behind the wait,
            // the stores and the proxy fence.  One lane per warp polls the stage's barrier and arrives for the warp.
            struct RowState {
                int ih0;
                unsigned col_mask;
                const unsigned *pix_base;     // window's first column in image row 0 (dereferenced only under the mask)
                bool row_ok;
            };
            auto row_state = [&](int tile) {
                int m_blk, n_blk;
                tile_coords(tile, p.m_tiles, p.n_tiles, m_blk, n_blk);
                const int m = m_blk * kBM + t;
                RowState rs;
                rs.row_ok = m < p.M;
                const int img = rs.row_ok ? m / (p.OH * p.OW) : 0;
                const int rem = rs.row_ok ? m - img * (p.OH * p.OW) : 0;
                const int oh = rem / p.OW, ow = rem - oh * p.OW;
                const int iw0 = ow * p.stride - p.pad;
                rs.ih0 = oh * p.stride - p.pad;
                rs.pix_base = reinterpret_cast<const unsigned *>(p.xe) + (int64_t)img * p.H * p.W + iw0;
                rs.col_mask = 0;
#pragma unroll
                for (int fs4 = 0; fs4 < 8; ++fs4)
                    if (fs4 < p.S && (unsigned)(iw0 + fs4) < (unsigned)p.W) rs.col_mask |= 1u << fs4;
                return rs;
            };
            auto load_rows = [&](const RowState &rs, int kb, unsigned (&v)[2][8]) {
#pragma unroll
                for (int j2 = 0; j2 < 2; ++j2) {
                    const int r = kb * 4 + half * 2 + j2;
                    const int ih = rs.ih0 + r;
                    const bool row_in = rs.row_ok && r < p.R && (unsigned)ih < (unsigned)p.H;
                    const unsigned *src_row = rs.pix_base + (int64_t)(row_in ? ih : 0) * p.W;
                    const unsigned mask = row_in ? rs.col_mask : 0u;
#pragma unroll
                    for (int w = 0; w < 8; ++w) v[j2][w] = ((mask >> w) & 1u) ? __ldg(src_row + w) : 0u;
                }
            };
            int tile = bid, kb = 0;
            if (tile < total_tiles) {
                RowState cur = row_state(tile);
                unsigned v[2][8], vn[2][8];
                load_rows(cur, 0, v);
                for (;; ++it) {
                    int ntile = tile, nkb = kb + 1;
                    if (nkb == p.k_blocks) {
                        nkb = 0;
                        ntile = tile + nblk;
                    }
                    const bool has_next = ntile < total_tiles;
                    if (has_next) {
                        if (ntile != tile) cur = row_state(ntile);      // (the current block's values are in v already)
                        load_rows(cur, nkb, vn);
                    }
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    bool got = true;
                    if ((threadIdx.x & 31) == 0) got = wait_bounded(&empty[s], ph ^ 1u, abort_flag, 5);
                    got = __shfl_sync(0xffffffffu, got, 0);
                    if (!got) break;
                    const uint32_t dst_row = smem_u32(a_stages + s * L::kAStage) + (uint32_t)t * kBKBytes;
#pragma unroll
                    for (int j2 = 0; j2 < 2; ++j2) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t dst = dst_row + (uint32_t)((((half * 2 + j2) * 2 + h) ^ sw) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v[j2][4 * h]),
                                         "r"(v[j2][4 * h + 1]), "r"(v[j2][4 * h + 2]), "r"(v[j2][4 * h + 3])
                                         : "memory");
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if ((threadIdx.x & 31) == 0) mbar_arrive(&full[s]);        // one arrival per warp
                    if (!has_next) break;
#pragma unroll
                    for (int j2 = 0; j2 < 2; ++j2)
#pragma unroll
                        for (int w = 0; w < 8; ++w) v[j2][w] = vn[j2][w];
                    tile = ntile;
                    kb = nkb;
                }
            }
        }
        for (int tile = bid; AMODE != kAGather4 && tile < total_tiles && ok; tile += nblk) {
            int m_blk, n_blk;
            tile_coords(tile, p.m_tiles, p.n_tiles, m_blk, n_blk);
            const int m = m_blk * kBM + t;
            const bool row_ok = m < p.M;
            const int img = row_ok ? m / (p.OH * p.OW) : 0;
            const int rem = row_ok ? m - img * (p.OH * p.OW) : 0;
            const int oh = rem / p.OW, ow = rem - oh * p.OW;
            const int ih0 = oh * p.stride - p.pad, iw0 = ow * p.stride - p.pad;
            const uint8_t *img_base = p.xe + (int64_t)img * p.H * p.W * p.cpb;
            // filter tap (fr, fs) and byte offset inside the pixel, advanced chunk by chunk: K runs (r, s, c)
            int fr = 0, fs = 0, cb = 0;
            for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                const int s = it % kStages;
                const uint32_t ph = (it / kStages) & 1u;
                if (!wait_bounded(&empty[s], ph ^ 1u, abort_flag, 5)) { ok = false; break; }
                const uint32_t dst_row = smem_u32(a_stages + s * L::kAStage) + (uint32_t)t * kBKBytes;
                if (AMODE == kAGather4) {
                    // handled above
                } else if (p.cpb % kBKBytes == 0) {
                    // a pixel holds whole 128-byte blocks: the eight chunks share one tap and are contiguous
                    const int ih = ih0 + fr * p.dil, iw = iw0 + fs * p.dil;
                    const bool in = row_ok && fr < p.R && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W;
                    const uint8_t *src = in ? img_base + ((int64_t)ih * p.W + iw) * p.cpb + cb : p.xe;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        cp_async_16(dst_row + (uint32_t)((j ^ sw) << 4), in ? src + j * 16 : src, in ? 16u : 0u);
                    cb += kBKBytes;
                    if (cb == p.cpb) {
                        cb = 0;
                        if (++fs == p.S) { fs = 0; ++fr; }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int ih = ih0 + fr * p.dil, iw = iw0 + fs * p.dil;
                        const bool in = row_ok && fr < p.R && (unsigned)ih < (unsigned)p.H && (unsigned)iw < (unsigned)p.W;
                        const uint8_t *src = in ? img_base + ((int64_t)ih * p.W + iw) * p.cpb + cb : p.xe;
                        cp_async_16(dst_row + (uint32_t)((j ^ sw) << 4), src, in ? 16u : 0u);
                        cb += 16;
                        if (cb == p.cpb) {
                            cb = 0;
                            if (++fs == p.S) { fs = 0; ++fr; }
                        }
                    }
                }
                cp_async_commit();
                ++issued;
                if (issued - published > kAhead) {
                    cp_async_wait_group<kAhead>();
                    fence_proxy_async_smem();
                    mbar_arrive(&full[published % kStages]);
                    ++published;
                }
            }
        }
        cp_async_wait_group<0>();
        fence_proxy_async_smem();
        while (ok && published < issued) {
            mbar_arrive(&full[published % kStages]);
            ++published;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (p.clock != nullptr && threadIdx.x == 32) atomicMax(p.clock + 1, (unsigned long long)global_timer_ns());
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <Kind KIND, int BN, int AMODE, int SWB>
__global__ void __launch_bounds__(AMODE == kAGather4 ? 576 : (AMODE == kAGather ? 448 : 320), 1)
dybit_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
    gemm_body<KIND, BN, AMODE, SWB>(tmap_a, tmap_b, tmap_c, p, (int)blockIdx.x, (int)gridDim.x);
}

// Several problems of one kernel configuration in ONE launch: CTAs [first_block[g], first_block[g + 1]) work on
// problem g exactly as the CTAs of a launch of its own would (same persistent tile loop over its own tiles).
constexpr int kMaxMulti = 16;
struct GemmMulti {
    int n;
    int first_block[kMaxMulti + 1];
    CUtensorMap ta[kMaxMulti], tb[kMaxMulti], tc[kMaxMulti];
    GemmParams p[kMaxMulti];
};

template <Kind KIND, int BN, int AMODE, int SWB>
__global__ void __launch_bounds__(320, 1) dybit_gemm_multi_kernel(const __grid_constant__ GemmMulti m) {
    int g = 0;
    while (g + 1 < m.n && (int)blockIdx.x >= m.first_block[g + 1]) ++g;
    gemm_body<KIND, BN, AMODE, SWB>(m.ta[g], m.tb[g], m.tc[g], m.p[g], (int)blockIdx.x - m.first_block[g],
                                    m.first_block[g + 1] - m.first_block[g]);
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static std::atomic<EncodeTiledFn> fn{nullptr};
    EncodeTiledFn f = fn.load(std::memory_order_acquire);
    if (f == nullptr) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess) {
            f = reinterpret_cast<EncodeTiledFn>(ptr);
            fn.store(f, std::memory_order_release);
        } else {
            (void)cudaGetLastError();
        }
    }
    return f;
}

// Byte matrix [rows][row_bytes] with row stride `stride`; box = swb bytes x box_rows, swb-byte swizzle.
static dybit_status make_operand_map(CUtensorMap *map, const void *base, int64_t rows, int64_t row_bytes, int64_t stride,
                                     int box_rows, int swb = 128) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return DYBIT_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)stride};
    cuuint32_t box[2] = {(cuuint32_t)swb, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DYBIT_OK : DYBIT_ERR_CUDA;
}

// Batched operand [batch][rows][row_bytes] (entries `bstride` bytes apart): box = 128 bytes x box_rows x 1 entry, so
// a tile never reaches into the next entry and rows past `rows` read as zeros.
static dybit_status make_operand_map_batched(CUtensorMap *map, const void *base, int64_t rows, int64_t row_bytes,
                                             int64_t stride, int64_t batch, int64_t bstride, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return DYBIT_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)row_bytes, (cuuint64_t)rows, (cuuint64_t)batch};
    cuuint64_t strides[2] = {(cuuint64_t)stride, (cuuint64_t)bstride};
    cuuint32_t box[3] = {128, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DYBIT_OK : DYBIT_ERR_CUDA;
}

typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeIm2colFn encode_im2col_fn() {
    static std::atomic<EncodeIm2colFn> fn{nullptr};
    EncodeIm2colFn f = fn.load(std::memory_order_acquire);
    if (f == nullptr) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess) {
            f = reinterpret_cast<EncodeIm2colFn>(ptr);
            fn.store(f, std::memory_order_release);
        } else {
            (void)cudaGetLastError();
        }
    }
    return f;
}

// Expanded activation [n][h][w][cpb bytes] as an im2col map: one load brings 128 consecutive output
// pixels x swb bytes of one filter tap, walking w, then h, then n with the convolution's stride and
// zero-filling taps outside the image.  The pixel box runs from -pad to pad - (filter - 1) * dilation.
static dybit_status make_im2col_map(CUtensorMap *map, const void *xe, const dybit_conv_desc *d, int64_t cpb, int swb) {
    EncodeIm2colFn fn = encode_im2col_fn();
    if (fn == nullptr) return DYBIT_ERR_CUDA;
    cuuint64_t dims[4] = {(cuuint64_t)cpb, (cuuint64_t)d->w, (cuuint64_t)d->h, (cuuint64_t)d->n};
    cuuint64_t strides[3] = {(cuuint64_t)cpb, (cuuint64_t)cpb * d->w, (cuuint64_t)cpb * d->w * d->h};
    int lower[2] = {-d->pad, -d->pad};
    int upper[2] = {d->pad - (d->s - 1) * d->dilation, d->pad - (d->r - 1) * d->dilation};
    cuuint32_t estr[4] = {1, (cuuint32_t)d->stride, (cuuint32_t)d->stride, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(xe), dims, strides, lower, upper,
                    (cuuint32_t)swb, (cuuint32_t)kBM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DYBIT_OK : DYBIT_ERR_CUDA;
}

// fp32 output [M][ldc] (batched: [batch][M][ldc] with `bstride` elements between entries) as a map whose box is
// 32 columns x 128 rows (x 1 entry), 128-byte swizzle (the staging layout).
static bool make_output_map(CUtensorMap *map, float *C, int64_t M, int64_t N, int64_t ldc, int64_t batch, int64_t bstride) {
    if ((reinterpret_cast<uintptr_t>(C) & 15) != 0 || (ldc * 4) % 16 != 0) return false;
    if (batch > 0 && (bstride * 4) % 16 != 0) return false;
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)(batch > 0 ? batch : 1)};
    cuuint64_t strides[2] = {(cuuint64_t)ldc * 4, (cuuint64_t)bstride * 4};
    cuuint32_t box[3] = {32, (cuuint32_t)kBM, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, batch > 0 ? 3 : 2, C, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor-core launches gathered instead of issued (dybit_conv2d_prepared_layers): problems that run on the same kernel
// configuration then share launches, up to kMaxMulti each.  One collector per host thread, active only inside that call.
struct MultiEntry {
    CUtensorMap ta, tb, tc;
    GemmParams p;
    unsigned char extra[512];      // the halo kernel's own parameter block (HaloParams) when fn launches that kernel
    int tiles, per_sm, smem;
    double work;                   // tiles x (K blocks + epilogue): the cost model behind the CTA shares
};
using MultiLaunchFn = dybit_status (*)(const MultiEntry *, int, cudaStream_t);
struct MultiGroup {
    MultiLaunchFn fn;
    int per_sm, smem;
    std::vector<MultiEntry> entries;
};
struct GemmCollector {
    std::vector<MultiGroup> groups;
    void add(MultiLaunchFn fn, const MultiEntry &e) {
        for (MultiGroup &g : groups)
            if (g.fn == fn && g.per_sm == e.per_sm && g.smem == e.smem) {
                g.entries.push_back(e);
                return;
            }
        groups.push_back(MultiGroup{fn, e.per_sm, e.smem, {e}});
    }
    dybit_status launch_all(cudaStream_t s) {
        for (const MultiGroup &g : groups)
            for (size_t i = 0; i < g.entries.size(); i += kMaxMulti) {
                const size_t n = g.entries.size() - i < (size_t)kMaxMulti ? g.entries.size() - i : (size_t)kMaxMulti;
                const dybit_status st = g.fn(g.entries.data() + i, (int)n, s);
                if (st != DYBIT_OK) return st;
            }
        return DYBIT_OK;
    }
};
inline GemmCollector *&gemm_collector() {
    static thread_local GemmCollector *c = nullptr;
    return c;
}

// CTAs of a shared launch.  If every tile of every problem can have a CTA of its own, it gets one.  Otherwise the
// `budget` CTAs the device holds at once are handed out one by one, each to the problem that would currently finish
// last (rounds of tiles per CTA x cost of a tile), so that whole rounds, not fractions, are balanced.
static void multi_shares(const MultiEntry *e, int n, int budget, int *first_block) {
    long long all_tiles = 0;
    for (int i = 0; i < n; ++i) all_tiles += e[i].tiles;
    int share[kMaxMulti];
    if (all_tiles <= budget) {
        for (int i = 0; i < n; ++i) share[i] = e[i].tiles;
    } else {
        for (int i = 0; i < n; ++i) share[i] = 1;
        for (int left = budget - n; left > 0; --left) {
            int worst = -1;
            double worst_t = -1.0;
            for (int i = 0; i < n; ++i) {
                if (share[i] >= e[i].tiles) continue;
                const double rounds = (double)((e[i].tiles + share[i] - 1) / share[i]);
                const double t = rounds * (e[i].work / (double)e[i].tiles);
                if (t > worst_t) {
                    worst_t = t;
                    worst = i;
                }
            }
            if (worst < 0) break;
            ++share[worst];
        }
    }
    first_block[0] = 0;
    for (int i = 0; i < n; ++i) first_block[i + 1] = first_block[i] + share[i];
}

template <Kind KIND, int BN, int AMODE, int SWB>
static dybit_status launch_gemm_multi(const MultiEntry *e, int n, cudaStream_t s) {
    using L = GemmSmem<BN, SWB>;
    auto kern = dybit_gemm_multi_kernel<KIND, BN, AMODE, SWB>;
    static std::atomic<bool> configured[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kBytes));
        configured[dev] = true;
    }
    GemmMulti m;
    memset(&m, 0, sizeof(m));
    m.n = n;
    multi_shares(e, n, sm_count(), m.first_block);
    for (int i = 0; i < n; ++i) {
        m.ta[i] = e[i].ta;
        m.tb[i] = e[i].tb;
        m.tc[i] = e[i].tc;
        m.p[i] = e[i].p;
        const int share = m.first_block[i + 1] - m.first_block[i];
        m.p[i].b_resident = (m.p[i].bmt == 0 && m.p[i].n_tiles == 1 && m.p[i].k_blocks <= L::kStages && e[i].tiles > share) ? 1 : 0;
    }
    launch_k(kern, dim3((unsigned)m.first_block[n]), dim3(320u), (size_t)L::kBytes, s, m);
    return launch_status();
}

template <Kind KIND, int BN, int AMODE, int SWB>
static dybit_status launch_gemm_inst(const CUtensorMap &ta, const CUtensorMap &tb, const GemmParams &p_in, cudaStream_t s) {
    GemmParams p = p_in;
    CUtensorMap tc;
    memset(&tc, 0, sizeof(tc));
    p.tma_store = (p.Q == nullptr && make_output_map(&tc, p.C, p.M, p.N, p.ldc, p.bmt ? p.m_tiles / p.bmt : 0, p.c_bstride)) ? 1 : 0;
    using L = GemmSmem<BN, SWB>;
    auto kern = dybit_gemm_kernel<KIND, BN, AMODE, SWB>;
    constexpr bool CONV = AMODE == kAGather || AMODE == kAGather4;
    static std::atomic<bool> configured[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kBytes));
        configured[dev] = true;
    }
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    ProfileEvents ev = profile_events();
    if constexpr (KIND == Kind::I8 && (AMODE == kAIm2col || AMODE == kATiled)) {
        // inside dybit_conv2d_prepared_layers: gathered, launched together with its like at the end of that call
        if (gemm_collector() != nullptr && !ev.start && !ev.stop && !ev.clock) {
            MultiEntry e;
            memset(&e, 0, sizeof(e));
            e.ta = ta;
            e.tb = tb;
            e.tc = tc;
            e.p = p;
            e.tiles = tiles;
            e.per_sm = 1;
            e.smem = L::kBytes;
            e.work = (double)tiles * (double)(p.k_blocks + 6);      // + a tile's epilogue, about six K blocks' worth (measured: 4-16 are within 8 %)
            gemm_collector()->add(launch_gemm_multi<KIND, BN, AMODE, SWB>, e);
            return DYBIT_OK;
        }
    }
    profile_events() = ProfileEvents();
    p.clock = ev.clock;
    // a B panel that fits the B stage slots is fetched once per CTA when every tile shares it and CTAs take several tiles
    p.b_resident = (!CONV && p.bmt == 0 && p.n_tiles == 1 && p.k_blocks <= L::kStages && tiles > sm_count()) ? 1 : 0;
    if (ev.start) DYBIT_CUDA_TRY(cudaEventRecord(ev.start, s));
    launch_k(kern, dim3((unsigned)(grid)), dim3((unsigned)(AMODE == kAGather4 ? 576 : (CONV ? 448 : 320))), (size_t)(L::kBytes), s, ta, tb,
             tc, p);
    const dybit_status st = launch_status();
    if (ev.stop) DYBIT_CUDA_TRY(cudaEventRecord(ev.stop, s));
    return st;
}

template <Kind KIND, int AMODE, int SWB>
static dybit_status launch_gemm_bn(int bn, const CUtensorMap &ta, const CUtensorMap &tb, const GemmParams &p,
                                   cudaStream_t s) {
    switch (bn) {
        case 64: return launch_gemm_inst<KIND, 64, AMODE, SWB>(ta, tb, p, s);
        case 128: return launch_gemm_inst<KIND, 128, AMODE, SWB>(ta, tb, p, s);
        default: return launch_gemm_inst<KIND, 256, AMODE, SWB>(ta, tb, p, s);
    }
}

template <int AMODE, int SWB>
static dybit_status launch_gemm_kind(dybit_container cont, int bn, const CUtensorMap &ta, const CUtensorMap &tb,
                                     const GemmParams &p, cudaStream_t s) {
    switch (cont) {
        case DYBIT_CONTAINER_I8: return launch_gemm_bn<Kind::I8, AMODE, SWB>(bn, ta, tb, p, s);
        case DYBIT_CONTAINER_E4M3: return launch_gemm_bn<Kind::F8F6F4, AMODE, SWB>(bn, ta, tb, p, s);
        default:
            if constexpr (AMODE == kAGather4) return DYBIT_ERR_UNSUPPORTED;     // one-byte elements only
            else return launch_gemm_bn<Kind::F16, AMODE, SWB>(bn, ta, tb, p, s);
    }
}

// Tile width along N: the narrowest of 64/128/256 that covers N, halved while that puts more SMs to work
// without opening a second, mostly empty wave: halve when the halved tiles still fit one wave, or when the
// current ones occupy less than half of the SMs.  (ResNet-18 layer 3 at batch 32, 49 x 1 tiles of 128 x 256:
// 98 tiles of 128 x 128 in one wave take 14.5 us, 196 tiles of 128 x 64 in two waves 20.3 us.)
static int choose_bn_tiles(int64_t m_tiles, int64_t N) {
    int bn = N <= 64 ? 64 : (N <= 128 ? 128 : 256);
    const int64_t sms = sm_count();
    while (bn > 64) {
        const int64_t tiles = m_tiles * ((N + bn - 1) / bn);
        const int64_t halved = m_tiles * ((N + bn / 2 - 1) / (bn / 2));
        if (tiles >= sms || !(halved <= sms || tiles * 2 < sms)) break;
        bn >>= 1;
    }
    return bn;
}

static int choose_bn(int64_t M, int64_t N) {
    // Launches that are shared between layers have tiles enough to fill the GPU, so a layer's tiles are not narrowed
    // to 64 columns to reach more SMs (a 64-wide instruction costs as much as a 128-wide one); 256-wide tiles gain
    // nothing over 128-wide ones there (measured on the ResNet-18 step: 153.8 / 164.0 us against 162.9 us narrowed).
    if (gemm_collector() != nullptr) return N <= 64 ? 64 : 128;
    return choose_bn_tiles((M + kBM - 1) / kBM, N);
}

static int pad_grid(int64_t chunks) {
    int64_t b = (chunks + 255) / 256, cap = (int64_t)sm_count() * 16;
    if (b > cap) b = cap;
    return b < 1 ? 1 : (int)b;
}

struct GemmLayout {
    dybit_container cont;
    int elem;
    int exp_a, exp_b;
    int64_t kp;             // K padded to 128 elements... in elements
    int64_t a_bytes, b_bytes, a_off, b_off, total;
};

static inline int64_t k_row_bytes(int64_t k_elems, int elem) { return round_up(k_elems * elem, kBKBytes); }

// Output of the re-quantizing entry points.
struct RequantSpec {
    dybit_fmt fq;
    const float *scale_q;
    const float *bias;
    int relu;
    void *Q;
    int64_t ldq;
};

static dybit_status check_requant(const RequantSpec *rq, int64_t N) {
    if (rq == nullptr) return DYBIT_OK;
    if (!fmt_ok(rq->fq) || rq->Q == nullptr || rq->scale_q == nullptr) return DYBIT_ERR_INVALID_ARG;
    if ((N * rq->fq.bits) % 8 != 0 || rq->ldq < N * rq->fq.bits / 8) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(rq->scale_q, 4) || !aligned(rq->bias, 4)) return DYBIT_ERR_ALIGNMENT;
    return DYBIT_OK;
}

static void apply_requant(GemmParams &p, const RequantSpec *rq) {
    if (rq == nullptr) return;
    p.Q = static_cast<uint8_t *>(rq->Q);
    p.ldq = rq->ldq;
    p.scale_q = rq->scale_q;
    p.q_bits = rq->fq.bits;
    p.q_signed = rq->fq.is_signed;
    p.relu = rq->relu;
    p.bias = rq->bias;
}

// How a convolution is lowered, and what it needs in the workspace.
enum ConvMode { kConvPointwise, kConvIm2col, kConvPix4, kConvPatch, kConvGather, kConvS2D };
struct ConvPlan {
    ConvMode mode;
    int elem, swb;
    int64_t cp, cpb, pixels;       // padded channels, bytes per pixel of the expanded activation
    int64_t a_bytes;               // first workspace region: expanded activation or patch matrix
    int64_t krow;                  // patch mode: bytes per patch row
    int64_t wrb;                   // bytes per expanded weight row
    bool pad_channels;             // expanded activation / weights carry zero channels c..cp-1
    int64_t xd_bytes;              // patch mode, dilation 1: dense container elements of the activation (third region)
    S2dGeom s2d;                   // kConvS2D
};

static ConvPlan plan_conv(const dybit_conv_desc *d, int oh, int ow, int elem) {
    ConvPlan c = {};
    c.elem = elem;
    c.cp = round_up(d->c, 16);
    c.cpb = c.cp * elem;
    c.pixels = (int64_t)d->n * d->h * d->w;
    const int64_t M = (int64_t)d->n * oh * ow;
    const int64_t taps = (int64_t)d->r * d->s;
    const bool pointwise = d->r == 1 && d->s == 1 && d->stride == 1 && d->pad == 0;
    // im2col TMA: a pixel must be a whole number of swizzle-span blocks, corners and tap offsets must fit the
    // descriptor's 8-bit fields, and the tensor must not be tiny
    c.swb = (c.cpb % 128 == 0) ? 128 : (c.cpb == 64 ? 64 : 0);
    const int up_w = d->pad - (d->s - 1) * d->dilation, up_h = d->pad - (d->r - 1) * d->dilation;
    const bool im2col_ok = c.swb != 0 && c.pixels * c.cpb >= 131072 && d->pad <= 127 && up_w >= -128 && up_h >= -128 &&
                           (d->s - 1) * d->dilation <= 255 && (d->r - 1) * d->dilation <= 255 && d->stride <= 8;
    const int64_t krow = round_up(taps * d->c * elem, 16);
    // at most four one-byte channels (the 3-channel stem): pixels become 32-bit words and the tensor-core kernel
    // gathers its A tile from them, four filter rows of eight taps per K block; no patch matrix is written
    const bool pix4_ok = elem == 1 && d->c <= 4 && d->dilation == 1 && d->s <= 8 && d->r <= 64;
    // stride 2 on at most four one-byte channels, even image sides, filter no wider than four rearranged taps (the
    // 3-channel 7 x 7 stem): 2 x 2 space-to-depth image + halo tiles (launch_conv_s2d)
    auto floordiv2 = [](int v) { return v >= 0 ? v / 2 : -((-v + 1) / 2); };
    S2dGeom g = {};
    g.lo_r = floordiv2(-d->pad);
    g.lo_s = g.lo_r;
    g.Rp = floordiv2(d->r - 1 - d->pad) - g.lo_r + 1;
    g.Sp = floordiv2(d->s - 1 - d->pad) - g.lo_s + 1;
    g.Hs = d->h / 2;
    g.Ws = d->w / 2;
    g.padL = -g.lo_s;
    g.P = g.padL + g.Ws + 3;
    const bool s2d_ok = elem == 1 && d->c <= 4 && d->stride == 2 && d->dilation == 1 && d->h % 2 == 0 && d->w % 2 == 0 &&
                        g.Rp >= 1 && g.Rp <= 4 && g.Sp >= 1 && g.Sp <= 4 && g.padL >= 0 && g.padL <= 2 && ow <= g.Ws + 1 &&
                        (int64_t)d->n * g.Hs * g.P * 16 < ((int64_t)1 << 40) && c.pixels < ((int64_t)1 << 31);
    if (pointwise) c.mode = kConvPointwise;
    else if (im2col_ok) c.mode = kConvIm2col;
    else if (s2d_ok) c.mode = kConvS2D;
    else if (pix4_ok) c.mode = kConvPix4;
    else if (krow <= 1024 && M * krow <= ((int64_t)1 << 32)) c.mode = kConvPatch;
    else c.mode = kConvGather;
    if (c.mode == kConvS2D) {
        c.s2d = g;
        c.a_bytes = round_up((int64_t)d->n * g.Hs * g.P * 16, 1024) + 1024;
        c.wrb = round_up((int64_t)g.Rp * 64, kBKBytes);
        c.pad_channels = false;
    } else if (c.mode == kConvPix4) {
        c.a_bytes = round_up(c.pixels * 4, 1024) + 1024;
        c.wrb = round_up((int64_t)d->r * 32, kBKBytes);
        c.pad_channels = false;
    } else if (c.mode == kConvPatch) {
        c.krow = krow;
        c.a_bytes = round_up(M * krow, 1024);
        c.wrb = k_row_bytes(taps * d->c, elem);
        c.pad_channels = false;
        if (d->dilation == 1) c.xd_bytes = round_up(round_up(c.pixels * d->c, kChunkCodes) * elem, 1024) + 1024;
    } else {
        c.a_bytes = round_up(c.pixels * c.cpb, 1024);
        c.wrb = k_row_bytes(taps * c.cp, elem);
        c.pad_channels = c.cp != d->c;
    }
    return c;
}

}  // namespace dybit

extern "C" {

size_t dybit_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, dybit_fmt fa, dybit_fmt fb) {
    using namespace dybit;
    ContainerPlan plan;
    if (M <= 0 || N <= 0 || K <= 0 || plan_container(fa, fb, &plan) != DYBIT_OK) return 0;
    const int elem = container_elem_bytes(plan.container);
    const int64_t rb = k_row_bytes(round_up(K, 128), elem);
    return (size_t)(round_up(M * rb, 1024) + round_up(N * rb, 1024) + 1024);
}

size_t dybit_gemm_batched_workspace_bytes(int64_t batch, int64_t M, int64_t N, int64_t K, dybit_fmt fa, dybit_fmt fb) {
    using namespace dybit;
    ContainerPlan plan;
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0 || plan_container(fa, fb, &plan) != DYBIT_OK) return 0;
    const int elem = container_elem_bytes(plan.container);
    const int64_t rb = k_row_bytes(round_up(K, 128), elem);
    return (size_t)(round_up(batch * M * rb, 1024) + round_up(batch * N * rb, 1024) + 1024);
}

size_t dybit_conv2d_workspace_bytes(const dybit_conv_desc *d, dybit_fmt fx, dybit_fmt fw) {
    using namespace dybit;
    ContainerPlan plan;
    int oh, ow;
    if (dybit_conv2d_out_hw(d, &oh, &ow) != DYBIT_OK || plan_container(fx, fw, &plan) != DYBIT_OK) return 0;
    const ConvPlan c = plan_conv(d, oh, ow, container_elem_bytes(plan.container));
    // expanded activation (or patch matrix), expanded weights, dense activation elements (patch mode), slack,
    // per-block maxima of the max-abs reduction
    return (size_t)(c.a_bytes + round_up((int64_t)d->k * c.wrb, 1024) + c.xd_bytes + 2048 + kMaxAbsmaxPartials * sizeof(unsigned));
}

}  // extern "C"

namespace dybit {

// CTA-pair variant of the plain GEMM (dybit_gemm_pair.cuh).
static bool gemm_pair_eligible(int64_t M, int64_t N, const GemmParams &p);
static dybit_status launch_gemm_pair(dybit_container cont, const void *ae, int64_t a_row_bytes, const void *be,
                                     int64_t b_row_bytes, int64_t M, int64_t N, const GemmParams &p_in, cudaStream_t s);

// Halo-tile lowering of stride-1 convolutions (dybit_conv_halo.cuh); DYBIT_ERR_UNSUPPORTED = not applicable.
static dybit_status launch_conv_halo(dybit_container cont, const dybit_conv_desc *d, int oh, int ow, int64_t cpb,
                                     const uint8_t *xe, const uint8_t *we, int64_t wrb, const GemmParams &p_in,
                                     cudaStream_t s);

// The GEMM that decodes its B operand in the main loop (dybit_gemm_bdec.cuh).
struct BdecTable {
    unsigned tab[4];          // the 16 table bytes of the 4-bit format, as expand4_lookup wants them
    int neg_high;
};
static std::atomic<int> &gemm_decode_mode();
static bool gemm_bdec_applicable(dybit_container cont, dybit_fmt fb, const ElemTable &tb, const GemmParams &p, BdecTable *bt);
static dybit_status launch_gemm_bdec(const uint8_t *ae, int64_t rb, const uint8_t *B, int64_t ldb_bytes, int64_t M, int64_t N,
                                     int64_t K, const GemmParams &p_in, const BdecTable &bt, cudaStream_t s);

static dybit_status launch_conv_s2d(dybit_container cont, const dybit_conv_desc *d, int oh, int ow, const S2dGeom &g,
                                    const uint8_t *xs, const uint8_t *we, int64_t wrb, const GemmParams &p_in,
                                    cudaStream_t s);

static dybit_status gemm_impl(int64_t M, int64_t N, int64_t K, const void *A, dybit_fmt fa, const float *scale_a,
                              int64_t lda_bytes, const void *B, dybit_fmt fb, const float *scale_b, int64_t ldb_bytes,
                              float *C, int64_t ldc, int32_t *C_raw, const RequantSpec *rq, void *ws, size_t ws_bytes,
                              void *stream) {
    if (M <= 0 || N <= 0 || K <= 0 || !fmt_ok(fa) || !fmt_ok(fb)) return DYBIT_ERR_INVALID_ARG;
    if (!A || !B || !scale_a || !scale_b) return DYBIT_ERR_INVALID_ARG;
    if (rq == nullptr && (!C || ldc < N)) return DYBIT_ERR_INVALID_ARG;
    {
        const dybit_status rs = check_requant(rq, N);
        if (rs != DYBIT_OK) return rs;
    }
    if (M > INT32_MAX - 256 || N > INT32_MAX - 256 || K > (1 << 24)) return DYBIT_ERR_UNSUPPORTED;
    if (lda_bytes < (int64_t)dybit_row_stride_bytes(K, fa.bits) || ldb_bytes < (int64_t)dybit_row_stride_bytes(K, fb.bits))
        return DYBIT_ERR_INVALID_ARG;
    if (lda_bytes % 16 || ldb_bytes % 16 || !aligned(A, 16) || !aligned(B, 16) || !aligned(C, 4) || !aligned(C_raw, 4) ||
        !aligned(scale_a, 4) || !aligned(scale_b, 4))
        return DYBIT_ERR_ALIGNMENT;
    ContainerPlan plan;
    dybit_status st = plan_container(fa, fb, &plan);
    if (st != DYBIT_OK) return st;
    if (C_raw && plan.container != DYBIT_CONTAINER_I8) return DYBIT_ERR_UNSUPPORTED;
    if (plan.container == DYBIT_CONTAINER_I8 && (K > (1 << 19) || K * plan.max_product > (int64_t)INT32_MAX))
        return DYBIT_ERR_UNSUPPORTED;
    const size_t need = dybit_gemm_workspace_bytes(M, N, K, fa, fb);
    if (!ws || ws_bytes < need) return DYBIT_ERR_WORKSPACE;
    if (!aligned(ws, 1024)) return DYBIT_ERR_ALIGNMENT;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int elem = container_elem_bytes(plan.container);
    const int64_t kp = round_up(K, 128);
    const int64_t rb = k_row_bytes(kp, elem);
    uint8_t *ae = static_cast<uint8_t *>(ws);
    uint8_t *be = ae + round_up(M * rb, 1024);
    const ElemTable &ta = make_elem_table(fa, plan.container, plan.exp_a);
    const ElemTable &tb = make_elem_table(fb, plan.container, plan.exp_b);
    const ExpandOperand opa = {static_cast<const uint8_t *>(A), fa.bits, M, lda_bytes, kp, ae, rb, &ta};
    const ExpandOperand opb = {static_cast<const uint8_t *>(B), fb.bits, N, ldb_bytes, kp, be, rb, &tb};
    const int bn = choose_bn(M, N);
    GemmParams p = {};
    p.M = (int)M;
    p.N = (int)N;
    p.k_blocks = (int)(rb / kBKBytes);
    p.m_tiles = (int)((M + kBM - 1) / kBM);
    p.n_tiles = (int)((N + bn - 1) / bn);
    p.C = C;
    p.C_raw = C_raw;
    p.ldc = ldc;
    p.scale_a = scale_a;
    p.scale_b = scale_b;
    p.pow2 = ldexp(1.0, -(plan.exp_a + plan.exp_b));
    apply_requant(p, rq);
    {
        // few rows of A against a long stream of 4-bit weights: leave the weights packed and decode them in the main
        // loop (0.5 byte of global traffic per weight instead of 2.5); only A goes through the expand pass
        const int mode = gemm_decode_mode().load(std::memory_order_relaxed);
        BdecTable bt_val = {};
        BdecTable *bt = &bt_val;
        if ((mode == 1 || (mode == 2 && M <= 128 && N * kp >= ((int64_t)1 << 25))) &&
            gemm_bdec_applicable(plan.container, fb, tb, p, bt)) {
            const ExpandOperand none = {static_cast<const uint8_t *>(B), fb.bits, 0, ldb_bytes, kp, be, rb, &tb};
            st = launch_expand_pair(opa, none, elem, true, s);
            if (st != DYBIT_OK) return st;
            st = launch_gemm_bdec(ae, rb, static_cast<const uint8_t *>(B), ldb_bytes, M, N, K, p, *bt, s);
            if (st != DYBIT_ERR_UNSUPPORTED) return st;
            // (the output cannot be described to the TMA: expand B as well and take the general kernel)
            const ExpandOperand only_b = {static_cast<const uint8_t *>(A), fa.bits, 0, lda_bytes, kp, ae, rb, &ta};
            st = launch_expand_pair(only_b, opb, elem, true, s);
            if (st != DYBIT_OK) return st;
        } else {
            st = launch_expand_pair(opa, opb, elem, plan.container == DYBIT_CONTAINER_I8, s);
            if (st != DYBIT_OK) return st;
        }
    }
    CUtensorMap map_a, map_b;
    st = make_operand_map(&map_a, ae, M, rb, rb, kBM);
    if (st != DYBIT_OK) return st;
    st = make_operand_map(&map_b, be, N, rb, rb, bn);
    if (st != DYBIT_OK) return st;
    if (gemm_pair_eligible(M, N, p)) {
        // large plain products: 256 x 256 tiles on pairs of SMs (falls through when C cannot be described to the TMA)
        st = launch_gemm_pair(plan.container, ae, rb, be, rb, M, N, p, s);
        if (st != DYBIT_ERR_UNSUPPORTED) return st;
    }
    return launch_gemm_kind<kATiled, 128>(plan.container, bn, map_a, map_b, p, s);
}

// Batched GEMM: `batch` independent products C_b = A_b * B_b^T of equal shape, one scale per operand tensor (the
// whole batch is one quantized tensor).  Every entry gets its own tiles: tile rows count over batch * m_tiles and
// the kernel's 3-D tensor maps keep a tile inside its entry.
static dybit_status gemm_batched_impl(int64_t batch, int64_t M, int64_t N, int64_t K, const void *A, dybit_fmt fa,
                                      const float *scale_a, int64_t lda_bytes, int64_t stride_a_bytes, const void *B,
                                      dybit_fmt fb, const float *scale_b, int64_t ldb_bytes, int64_t stride_b_bytes,
                                      float *C, int64_t ldc, int64_t stride_c, int32_t *C_raw, void *ws, size_t ws_bytes,
                                      void *stream) {
    if (batch <= 0 || M <= 0 || N <= 0 || K <= 0 || !fmt_ok(fa) || !fmt_ok(fb)) return DYBIT_ERR_INVALID_ARG;
    if (!A || !B || !scale_a || !scale_b || !C || ldc < N || stride_c < (M - 1) * ldc + N) return DYBIT_ERR_INVALID_ARG;
    if (M > (1 << 24) || N > (1 << 24) || K > (1 << 24) || batch > (1 << 24)) return DYBIT_ERR_UNSUPPORTED;
    const int64_t m_tiles = (M + kBM - 1) / kBM;
    if (batch * m_tiles > (1 << 24)) return DYBIT_ERR_UNSUPPORTED;
    if (lda_bytes < (int64_t)dybit_row_stride_bytes(K, fa.bits) || ldb_bytes < (int64_t)dybit_row_stride_bytes(K, fb.bits) ||
        stride_a_bytes < M * lda_bytes || stride_b_bytes < N * ldb_bytes)
        return DYBIT_ERR_INVALID_ARG;
    if (lda_bytes % 16 || ldb_bytes % 16 || stride_a_bytes % 16 || stride_b_bytes % 16 || !aligned(A, 16) || !aligned(B, 16) ||
        !aligned(C, 4) || !aligned(C_raw, 4) || !aligned(scale_a, 4) || !aligned(scale_b, 4))
        return DYBIT_ERR_ALIGNMENT;
    ContainerPlan plan;
    dybit_status st = plan_container(fa, fb, &plan);
    if (st != DYBIT_OK) return st;
    if (C_raw && plan.container != DYBIT_CONTAINER_I8) return DYBIT_ERR_UNSUPPORTED;
    if (plan.container == DYBIT_CONTAINER_I8 && (K > (1 << 19) || K * plan.max_product > (int64_t)INT32_MAX))
        return DYBIT_ERR_UNSUPPORTED;
    const size_t need = dybit_gemm_batched_workspace_bytes(batch, M, N, K, fa, fb);
    if (need == 0) return DYBIT_ERR_INVALID_ARG;
    if (!ws || ws_bytes < need) return DYBIT_ERR_WORKSPACE;
    if (!aligned(ws, 1024)) return DYBIT_ERR_ALIGNMENT;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int elem = container_elem_bytes(plan.container);
    const int64_t kp = round_up(K, 128);
    const int64_t rb = k_row_bytes(kp, elem);
    uint8_t *ae = static_cast<uint8_t *>(ws);
    uint8_t *be = ae + round_up(batch * M * rb, 1024);
    const ElemTable &ta = make_elem_table(fa, plan.container, plan.exp_a);
    const ElemTable &tb = make_elem_table(fb, plan.container, plan.exp_b);
    const bool i8 = plan.container == DYBIT_CONTAINER_I8;
    if (stride_a_bytes == M * lda_bytes && stride_b_bytes == N * ldb_bytes) {
        // dense batches: all entries of an operand are one run of rows
        const ExpandOperand opa = {static_cast<const uint8_t *>(A), fa.bits, batch * M, lda_bytes, kp, ae, rb, &ta};
        const ExpandOperand opb = {static_cast<const uint8_t *>(B), fb.bits, batch * N, ldb_bytes, kp, be, rb, &tb};
        st = launch_expand_pair(opa, opb, elem, i8, s);
        if (st != DYBIT_OK) return st;
    } else {
        for (int64_t b = 0; b < batch; ++b) {
            const ExpandOperand opa = {static_cast<const uint8_t *>(A) + b * stride_a_bytes, fa.bits, M, lda_bytes, kp,
                                       ae + b * M * rb, rb, &ta};
            const ExpandOperand opb = {static_cast<const uint8_t *>(B) + b * stride_b_bytes, fb.bits, N, ldb_bytes, kp,
                                       be + b * N * rb, rb, &tb};
            st = launch_expand_pair(opa, opb, elem, i8, s);
            if (st != DYBIT_OK) return st;
        }
    }
    const int bn = choose_bn(batch * m_tiles * kBM, N);
    CUtensorMap map_a, map_b;
    st = make_operand_map_batched(&map_a, ae, M, rb, rb, batch, M * rb, kBM);
    if (st != DYBIT_OK) return st;
    st = make_operand_map_batched(&map_b, be, N, rb, rb, batch, N * rb, bn);
    if (st != DYBIT_OK) return st;
    GemmParams p = {};
    p.M = (int)M;
    p.N = (int)N;
    p.k_blocks = (int)(rb / kBKBytes);
    p.bmt = (int)m_tiles;
    p.m_tiles = (int)(batch * m_tiles);
    p.n_tiles = (int)((N + bn - 1) / bn);
    p.C = C;
    p.C_raw = C_raw;
    p.ldc = ldc;
    p.c_bstride = stride_c;
    p.scale_a = scale_a;
    p.scale_b = scale_b;
    p.pow2 = ldexp(1.0, -(plan.exp_a + plan.exp_b));
    return launch_gemm_kind<kATiled, 128>(plan.container, bn, map_a, map_b, p, s);
}

// An fp32 activation to quantize on the way in (dybit_quantize_conv2d): X then is the buffer that receives its
// packed codes and scale_x the pair the codes are made with (written first when `given` is null).
struct QuantInput {
    const float *x;
    const float *given;       // scale to use, or null for the max-abs scale
};

static dybit_status conv_impl(const dybit_conv_desc *d, const void *X, dybit_fmt fx, const float *scale_x, const void *W,
                              dybit_fmt fw, const float *scale_w, int64_t ldw_bytes, float *Y, int32_t *Y_raw,
                              const RequantSpec *rq, void *ws, size_t ws_bytes, void *stream,
                              const QuantInput *xq = nullptr, LayerCollector *col = nullptr, bool prepared = false) {
    int oh, ow;
    dybit_status st = dybit_conv2d_out_hw(d, &oh, &ow);
    if (st != DYBIT_OK) return st;
    if (!fmt_ok(fx) || !fmt_ok(fw) || !X || !W || !scale_x || !scale_w) return DYBIT_ERR_INVALID_ARG;
    if (xq && (!xq->x || !aligned(xq->x, 4) || !aligned(xq->given, 4))) return xq->x ? DYBIT_ERR_ALIGNMENT : DYBIT_ERR_INVALID_ARG;
    if (rq == nullptr && !Y) return DYBIT_ERR_INVALID_ARG;
    {
        const dybit_status rs = check_requant(rq, d->k);
        if (rs != DYBIT_OK) return rs;
    }
    const int64_t K = (int64_t)d->r * d->s * d->c;
    const int64_t M = (int64_t)d->n * oh * ow;
    const int64_t N = d->k;
    if (M > INT32_MAX - 256 || K > (1 << 24)) return DYBIT_ERR_UNSUPPORTED;
    if (ldw_bytes < (int64_t)dybit_row_stride_bytes(K, fw.bits)) return DYBIT_ERR_INVALID_ARG;
    if (ldw_bytes % 16 || !aligned(X, 16) || !aligned(W, 16) || !aligned(Y, 4) || !aligned(Y_raw, 4) ||
        !aligned(scale_x, 4) || !aligned(scale_w, 4))
        return DYBIT_ERR_ALIGNMENT;
    ContainerPlan plan;
    st = plan_container(fx, fw, &plan);
    if (st != DYBIT_OK) return st;
    if (Y_raw && plan.container != DYBIT_CONTAINER_I8) return DYBIT_ERR_UNSUPPORTED;
    if (plan.container == DYBIT_CONTAINER_I8 && (K > (1 << 19) || K * plan.max_product > (int64_t)INT32_MAX))
        return DYBIT_ERR_UNSUPPORTED;
    const size_t need = dybit_conv2d_workspace_bytes(d, fx, fw);
    if (!ws || ws_bytes < need) return DYBIT_ERR_WORKSPACE;
    if (!aligned(ws, 1024)) return DYBIT_ERR_ALIGNMENT;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int elem = container_elem_bytes(plan.container);
    const ConvPlan cv = plan_conv(d, oh, ow, elem);
    const int64_t cp = cv.cp, pixels = cv.pixels, wrb = cv.wrb;
    uint8_t *xe = static_cast<uint8_t *>(ws);
    uint8_t *we = xe + cv.a_bytes;
    uint8_t *xd = we + round_up(N * wrb, 1024);              // patch mode: dense container elements of the activation
    const bool patch_dense = cv.mode == kConvPatch && cv.xd_bytes > 0;
    const bool s2d = cv.mode == kConvS2D;
    const bool pix4 = cv.mode == kConvPix4 || s2d;           // pixels of <= 4 one-byte channels, written pixel by pixel
    FusedWeights wpix = {static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, wrb, we, wrb, 0, {}, d->c, d->r, d->s,
                         s2d ? 1 : 0, cv.s2d.lo_r, cv.s2d.lo_s, d->pad, cv.s2d.Rp};
    PixLayout pl = {};
    if (s2d) pl = PixLayout{d->c, 1, d->h, d->w, cv.s2d.Hs, cv.s2d.P, cv.s2d.padL};
    else if (pix4 && d->c < 4) pl.c = d->c;                  // four channels: the code order is the pixel-word layout already
    const ElemTable &tx = make_elem_table(fx, plan.container, plan.exp_a);
    const ElemTable &tw = make_elem_table(fw, plan.container, plan.exp_b);
    const bool i8 = plan.container == DYBIT_CONTAINER_I8;
    bool expanded = false;
    // `col`: the layer's max-abs and quantize + expand work is only gathered here (several layers then share a
    // launch) and the call ends there; `prepared`: that work has been done, only what follows it is launched.
    // Both need the lowering whose quantize launch also writes the expanded operands.
    const bool fused_lowering = patch_dense || pix4 || (cv.mode != kConvPatch && !cv.pad_channels);
    if ((col || prepared) && (!xq || !fused_lowering || pixels * d->c <= 0)) return DYBIT_ERR_UNSUPPORTED;
    if (prepared) {
        expanded = true;
    } else if (xq) {
        // scale first (max-abs, or a copy of the given pair), then codes; where the expanded activation is the code
        // order itself, one launch writes the codes, their container elements and the expanded weights
        const int64_t n_x = pixels * d->c;
        float *scale_dst = const_cast<float *>(scale_x);
        const bool fused = fused_lowering;
        // max-abs scale: in the fused case the absmax launch leaves one maximum per block in the workspace and the
        // quantize launch folds them (nothing to zero first, no atomics); otherwise the ticket version writes the pair
        unsigned *partials = nullptr;
        int n_partials = 0;
        if (xq->given == nullptr && fused && n_x > 0) {
            partials = reinterpret_cast<unsigned *>(static_cast<uint8_t *>(ws) + need - kMaxAbsmaxPartials * sizeof(unsigned));
            st = col ? col->add_absmax(xq->x, n_x, partials, &n_partials)
                     : launch_absmax(xq->x, 1, n_x, n_x, fx, scale_dst, s, partials, &n_partials);
            if (st != DYBIT_OK) return st;
        } else if (xq->given == nullptr) {
            st = launch_absmax(xq->x, 1, n_x, n_x, fx, scale_dst, s);
            if (st != DYBIT_OK) return st;
        } else if (xq->given != scale_x) {
            DYBIT_CUDA_TRY(cudaMemcpyAsync(scale_dst, xq->given, 2 * sizeof(float), cudaMemcpyDeviceToDevice, s));
        }
        uint8_t *packed = static_cast<uint8_t *>(const_cast<void *>(X));
        const int64_t packed_bytes = (int64_t)dybit_packed_bytes(n_x, fx.bits);
        if (fused) {
            FusedWeights wj = {static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, wrb / elem, we, wrb, 0, {}, 0, 0, 0};
            const ExpandOperand opw = {static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, wrb / elem, we, wrb, &tw};
            wj.use4 = expand4_job(opw, elem, i8, &wj.job4) ? 1 : 0;
            if (pix4) wj = wpix;
            XTab4 xt = {};
            {
                Expand4Job xj;
                const ExpandOperand opx = {packed, fx.bits, 1, 0, 32, xe, 0, &tx};
                if (expand4_job(opx, elem, i8, &xj)) {
                    for (int i = 0; i < 4; ++i) xt.tab[i] = xj.tab[i];
                    xt.use = 1;
                    xt.neg_high = xj.neg_high;
                }
            }
            uint8_t *const dense = patch_dense ? xd : xe;         // code order either way
            const int64_t dense_bytes = patch_dense ? cv.xd_bytes : cv.a_bytes;
            QeLaunch one = nullptr;
            QeLayersLaunch many = nullptr;
            if (!(elem == 1 ? qe_launchers<1>(fx, &one, &many) : qe_launchers<2>(fx, &one, &many))) return DYBIT_ERR_INVALID_ARG;
            int blocks = 0;
            const QeArgs qa = make_qe_args(xq->x, n_x, fx, elem, scale_x, packed, packed_bytes, dense, dense_bytes, wj, partials,
                                           n_partials, scale_dst, elem == 1 ? pl : PixLayout{}, col == nullptr, &blocks);
            if (col) return col->add_qe(fx, fw, elem, tx, tw, xt, many, qa, blocks);
            st = one(qa, blocks, tx, tw, xt, s);
            if (st != DYBIT_OK) return st;
            expanded = true;
        } else {
            st = launch_quantize(xq->x, 1, n_x, n_x, fx, scale_x, packed, packed_bytes, s);
            if (st != DYBIT_OK) return st;
        }
    }
    if (pix4) {
        if (!expanded) {
            // pixels to 32-bit words and the weights to filter rows of eight taps, in one launch
            int64_t x_blocks = (pixels + 256 * 8 - 1) / (256 * 8), w_blocks = (N * (wrb / 16) + 1023) / 1024;
            if (x_blocks > (int64_t)sm_count() * 8) x_blocks = (int64_t)sm_count() * 8;
            if (w_blocks > sm_count()) w_blocks = sm_count();
            launch_k(expand_pix4_kernel, dim3((unsigned)(x_blocks + w_blocks)), dim3(256u), (size_t)0, s,
                     static_cast<const uint8_t *>(X), fx.bits, pixels, d->c, reinterpret_cast<unsigned *>(xe), tx, wpix, tw,
                     (int)x_blocks, pl);
            if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
        }
    } else if (patch_dense) {
        // dense container elements first (unless the quantize launch wrote them), then the patch matrix from those
        if (!expanded) {
            const int64_t n_codes = pixels * d->c;
            const ExpandOperand opx = {static_cast<const uint8_t *>(X), fx.bits, 1, 0,
                                       fx.bits == 4 ? round_up(n_codes, 32) : n_codes, xd, 0, &tx};
            const ExpandOperand opw = {static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, wrb / elem, we, wrb, &tw};
            st = launch_expand_pair(opx, opw, elem, i8, s);
            if (st != DYBIT_OK) return st;
        }
        PatchGatherParams pg = {};
        pg.xd = xd;
        pg.out = xe;
        pg.elem = elem;
        pg.H = d->h; pg.W = d->w; pg.C = d->c; pg.R = d->r; pg.S = d->s;
        pg.OH = oh; pg.OW = ow; pg.stride = d->stride; pg.pad = d->pad;
        pg.M = (int)M;
        pg.krow = (int)cv.krow;
        pg.row_pitch = (int)cv.krow + 4;
        const size_t smem = (size_t)128 * pg.row_pitch;
        static std::atomic<bool> gather_configured[64];
        int dev = 0;
        DYBIT_CUDA_TRY(cudaGetDevice(&dev));
        if (dev >= 0 && dev < 64 && !gather_configured[dev]) {
            DYBIT_CUDA_TRY(cudaFuncSetAttribute(patch_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                128 * (1024 + 4)));
            gather_configured[dev] = true;
        }
        launch_k(patch_gather_kernel, dim3((unsigned)((int)((M + 127) / 128))), dim3((unsigned)(128)), (size_t)(smem), s, pg);
        if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
    } else if (expanded) {
        // nothing left to expand
    } else if (cv.mode == kConvPatch) {
        // patch matrix from the packed activation in one kernel; weights expand as plain rows (K order r, s, c)
        PatchParams pp = {};
        pp.packed = static_cast<const uint8_t *>(X);
        pp.packed_words = (int64_t)dybit_packed_bytes(pixels * d->c, fx.bits) / 4;
        pp.out = xe;
        pp.bits = fx.bits;
        pp.elem = elem;
        pp.H = d->h; pp.W = d->w; pp.C = d->c; pp.R = d->r; pp.S = d->s;
        pp.OH = oh; pp.OW = ow; pp.stride = d->stride; pp.pad = d->pad; pp.dil = d->dilation;
        pp.M = (int)M;
        pp.krow = (int)cv.krow;
        pp.row_pitch = (int)cv.krow + 4;
        const size_t smem = (size_t)128 * pp.row_pitch;
        static std::atomic<bool> patch_configured[64];
        int dev = 0;
        DYBIT_CUDA_TRY(cudaGetDevice(&dev));
        if (dev >= 0 && dev < 64 && !patch_configured[dev]) {
            DYBIT_CUDA_TRY(cudaFuncSetAttribute(patch_expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                128 * (1024 + 4)));
            patch_configured[dev] = true;
        }
        launch_k(patch_expand_kernel, dim3((unsigned)((int)((M + 127) / 128))), dim3((unsigned)(128)), (size_t)(smem), s, pp, tx);
        if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
        st = launch_expand(static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, wrb / elem, elem, we, wrb, tw, s);
        if (st != DYBIT_OK) return st;
    } else if (!cv.pad_channels) {
        // channels already a multiple of 16: X is one flat run, W rows expand with their zero tail
        const ExpandOperand opx = {static_cast<const uint8_t *>(X), fx.bits, 1, 0, pixels * cp, xe, 0, &tx};
        const ExpandOperand opw = {static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, wrb / elem, we, wrb, &tw};
        st = launch_expand_pair(opx, opw, elem, i8, s);
        if (st != DYBIT_OK) return st;
    } else {
        const int64_t taps = (int64_t)d->r * d->s;
        DYBIT_CUDA_TRY(cudaMemsetAsync(we, 0, (size_t)(N * wrb), s));
        int64_t chunks = pixels * (cp * elem / 16);
        launch_k(expand_pad_kernel, dim3((unsigned)(pad_grid(chunks))), dim3((unsigned)(256)), (size_t)(0), s, 
            static_cast<const uint8_t *>(X), fx.bits, 1, 0, pixels, d->c, (int)cp, elem, xe, 0, tx);
        if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
        chunks = N * taps * (cp * elem / 16);
        launch_k(expand_pad_kernel, dim3((unsigned)(pad_grid(chunks))), dim3((unsigned)(256)), (size_t)(0), s, 
            static_cast<const uint8_t *>(W), fw.bits, N, ldw_bytes, taps, d->c, (int)cp, elem, we, wrb, tw);
        if (launch_status() != DYBIT_OK) return DYBIT_ERR_CUDA;
    }

    const int bn = choose_bn(M, N);
    const int64_t cpb = cp * elem;
    GemmParams p = {};
    p.M = (int)M;
    p.N = (int)N;
    p.m_tiles = (int)((M + kBM - 1) / kBM);
    p.n_tiles = (int)((N + bn - 1) / bn);
    p.C = Y;
    p.C_raw = Y_raw;
    p.ldc = N;
    p.scale_a = scale_x;
    p.scale_b = scale_w;
    p.pow2 = ldexp(1.0, -(plan.exp_a + plan.exp_b));
    p.xe = xe;
    p.H = d->h;
    p.W = d->w;
    p.OH = oh;
    p.OW = ow;
    p.R = d->r;
    p.S = d->s;
    p.stride = d->stride;
    p.pad = d->pad;
    p.dil = d->dilation;
    p.cpb = (int)cpb;
    apply_requant(p, rq);

    CUtensorMap map_a, map_b;
    if (cv.mode == kConvPointwise || cv.mode == kConvPatch) {
        // a GEMM on a row-major A: the expanded activation itself (1x1, stride 1) or the patch matrix
        const int64_t arow = cv.mode == kConvPatch ? cv.krow : cpb;
        st = make_operand_map(&map_a, xe, M, arow, arow, kBM);
        if (st != DYBIT_OK) return st;
        st = make_operand_map(&map_b, we, N, wrb, wrb, bn);
        if (st != DYBIT_OK) return st;
        p.k_blocks = (int)(wrb / kBKBytes);
        if (gemm_pair_eligible(M, N, p)) {
            st = launch_gemm_pair(plan.container, xe, arow, we, wrb, M, N, p, s);
            if (st != DYBIT_ERR_UNSUPPORTED) return st;
        }
        return launch_gemm_kind<kATiled, 128>(plan.container, bn, map_a, map_b, p, s);
    }
    if (cv.mode == kConvIm2col || cv.mode == kConvGather) {
        // stride 1, filters up to three rows, pixels of 64 or k * 128 bytes: halo tiles (every pixel fetched S times
        // instead of R * S times); same workspace layout as the two lowerings below
        st = launch_conv_halo(plan.container, d, oh, ow, cpb, xe, we, wrb, p, s);
        if (st != DYBIT_ERR_UNSUPPORTED) return st;
    }
    if (cv.mode == kConvIm2col) {
        const int swb = cv.swb;
        st = make_im2col_map(&map_a, xe, d, cpb, swb);
        if (st != DYBIT_OK) return st;
        st = make_operand_map(&map_b, we, N, wrb, wrb, bn, swb);
        if (st != DYBIT_OK) return st;
        p.kb_per_tap = (int)(cpb / swb);
        p.k_blocks = (int)((int64_t)d->r * d->s * p.kb_per_tap);
        return swb == 128 ? launch_gemm_kind<kAIm2col, 128>(plan.container, bn, map_a, map_b, p, s)
                          : launch_gemm_kind<kAIm2col, 64>(plan.container, bn, map_a, map_b, p, s);
    }
    if (s2d) return launch_conv_s2d(plan.container, d, oh, ow, cv.s2d, xe, we, wrb, p, s);
    st = make_operand_map(&map_b, we, N, wrb, wrb, bn);
    if (st != DYBIT_OK) return st;
    p.k_blocks = (int)(wrb / kBKBytes);
    if (pix4) return launch_gemm_kind<kAGather4, 128>(plan.container, bn, map_b, map_b, p, s);
    return launch_gemm_kind<kAGather, 128>(plan.container, bn, map_b, map_b, p, s);
}

}  // namespace dybit

extern "C" {

dybit_status dybit_selftest_wait_timeout(uint64_t limit_ns, uint32_t *result, void *stream) {
    if (result == nullptr || limit_ns == 0 || limit_ns > 100000000ull) return DYBIT_ERR_INVALID_ARG;   // at most 0.1 s
    if (!dybit::aligned(result, 4)) return DYBIT_ERR_ALIGNMENT;
    dybit::launch_k(dybit::wait_timeout_selftest_kernel, dim3(1u), dim3(32u), (size_t)0, static_cast<cudaStream_t>(stream),
                    (unsigned long long)limit_ns, result);
    return dybit::launch_status();
}

dybit_status dybit_gemm(int64_t M, int64_t N, int64_t K, const void *A, dybit_fmt fa, const float *scale_a,
                        int64_t lda_bytes, const void *B, dybit_fmt fb, const float *scale_b, int64_t ldb_bytes,
                        float *C, int64_t ldc, int32_t *C_raw, void *ws, size_t ws_bytes, void *stream) {
    return dybit::gemm_impl(M, N, K, A, fa, scale_a, lda_bytes, B, fb, scale_b, ldb_bytes, C, ldc, C_raw, nullptr, ws,
                            ws_bytes, stream);
}

dybit_status dybit_gemm_batched(int64_t batch, int64_t M, int64_t N, int64_t K, const void *A, dybit_fmt fa,
                                const float *scale_a, int64_t lda_bytes, int64_t stride_a_bytes, const void *B,
                                dybit_fmt fb, const float *scale_b, int64_t ldb_bytes, int64_t stride_b_bytes, float *C,
                                int64_t ldc, int64_t stride_c, int32_t *C_raw, void *ws, size_t ws_bytes, void *stream) {
    return dybit::gemm_batched_impl(batch, M, N, K, A, fa, scale_a, lda_bytes, stride_a_bytes, B, fb, scale_b, ldb_bytes,
                                    stride_b_bytes, C, ldc, stride_c, C_raw, ws, ws_bytes, stream);
}

dybit_status dybit_conv2d(const dybit_conv_desc *d, const void *X, dybit_fmt fx, const float *scale_x, const void *W,
                          dybit_fmt fw, const float *scale_w, int64_t ldw_bytes, float *Y, int32_t *Y_raw, void *ws,
                          size_t ws_bytes, void *stream) {
    return dybit::conv_impl(d, X, fx, scale_x, W, fw, scale_w, ldw_bytes, Y, Y_raw, nullptr, ws, ws_bytes, stream);
}

dybit_status dybit_quantize_conv2d(const dybit_conv_desc *d, const float *X, dybit_fmt fx, const float *scale_x,
                                   float *scale_x_out, void *X_packed, const void *W, dybit_fmt fw, const float *scale_w,
                                   int64_t ldw_bytes, float *Y, int32_t *Y_raw, void *ws, size_t ws_bytes, void *stream) {
    if (scale_x_out == nullptr || X_packed == nullptr) return DYBIT_ERR_INVALID_ARG;
    const dybit::QuantInput xq = {X, scale_x};
    return dybit::conv_impl(d, X_packed, fx, scale_x_out, W, fw, scale_w, ldw_bytes, Y, Y_raw, nullptr, ws, ws_bytes, stream, &xq);
}

dybit_status dybit_quantize_expand_layers(const dybit_conv_layer *layers, int n_layers, void *stream) {
    if (layers == nullptr || n_layers <= 0) return DYBIT_ERR_INVALID_ARG;
    dybit::LayerCollector col;
    for (int i = 0; i < n_layers; ++i) {
        const dybit_conv_layer &l = layers[i];
        if (l.scale_x_out == nullptr || l.X_packed == nullptr) return DYBIT_ERR_INVALID_ARG;
        const dybit::QuantInput xq = {l.X, l.scale_x};
        const dybit::RequantSpec rq = {l.fq, l.scale_q, l.bias, l.relu ? 1 : 0, l.Q, (int64_t)l.desc.k * l.fq.bits / 8};
        const dybit_status st = dybit::conv_impl(&l.desc, l.X_packed, l.fx, l.scale_x_out, l.W, l.fw, l.scale_w, l.ldw_bytes,
                                                 l.Q ? nullptr : l.Y, l.Q ? nullptr : l.Y_raw, l.Q ? &rq : nullptr, l.ws,
                                                 l.ws_bytes, stream, &xq, &col, false);
        if (st != DYBIT_OK) return st;
    }
    return col.launch_all(static_cast<cudaStream_t>(stream));
}

dybit_status dybit_conv2d_prepared(const dybit_conv_layer *layer, void *stream) {
    if (layer == nullptr || layer->scale_x_out == nullptr || layer->X_packed == nullptr) return DYBIT_ERR_INVALID_ARG;
    const dybit_conv_layer &l = *layer;
    const dybit::QuantInput xq = {l.X, l.scale_x};
    const dybit::RequantSpec rq = {l.fq, l.scale_q, l.bias, l.relu ? 1 : 0, l.Q, (int64_t)l.desc.k * l.fq.bits / 8};
    if (l.Q != nullptr && l.Y_raw != nullptr) return DYBIT_ERR_INVALID_ARG;
    return dybit::conv_impl(&l.desc, l.X_packed, l.fx, l.scale_x_out, l.W, l.fw, l.scale_w, l.ldw_bytes, l.Q ? nullptr : l.Y,
                            l.Q ? nullptr : l.Y_raw, l.Q ? &rq : nullptr, l.ws, l.ws_bytes, stream, &xq, nullptr, true);
}

dybit_status dybit_conv2d_prepared_layers(const dybit_conv_layer *layers, int n_layers, void *stream) {
    if (layers == nullptr || n_layers <= 0) return DYBIT_ERR_INVALID_ARG;
    dybit::GemmCollector col;
    dybit::gemm_collector() = &col;
    dybit_status st = DYBIT_OK;
    for (int i = 0; i < n_layers && st == DYBIT_OK; ++i) st = dybit_conv2d_prepared(&layers[i], stream);
    dybit::gemm_collector() = nullptr;
    if (st != DYBIT_OK) return st;
    return col.launch_all(static_cast<cudaStream_t>(stream));
}

dybit_status dybit_gemm_requant(int64_t M, int64_t N, int64_t K, const void *A, dybit_fmt fa, const float *scale_a,
                                int64_t lda_bytes, const void *B, dybit_fmt fb, const float *scale_b,
                                int64_t ldb_bytes, dybit_fmt fq, const float *scale_q, const float *bias, int relu, void *Q,
                                int64_t ldq_bytes, void *ws, size_t ws_bytes, void *stream) {
    const dybit::RequantSpec rq = {fq, scale_q, bias, relu ? 1 : 0, Q, ldq_bytes};
    return dybit::gemm_impl(M, N, K, A, fa, scale_a, lda_bytes, B, fb, scale_b, ldb_bytes, nullptr, 0, nullptr, &rq, ws,
                            ws_bytes, stream);
}

dybit_status dybit_conv2d_requant(const dybit_conv_desc *d, const void *X, dybit_fmt fx, const float *scale_x,
                                  const void *W, dybit_fmt fw, const float *scale_w, int64_t ldw_bytes, dybit_fmt fq,
                                  const float *scale_q, const float *bias, int relu, void *Q, void *ws,
                                  size_t ws_bytes, void *stream) {
    if (d == nullptr) return DYBIT_ERR_INVALID_ARG;
    const dybit::RequantSpec rq = {fq, scale_q, bias, relu ? 1 : 0, Q, (int64_t)d->k * fq.bits / 8};
    return dybit::conv_impl(d, X, fx, scale_x, W, fw, scale_w, ldw_bytes, nullptr, nullptr, &rq, ws, ws_bytes, stream);
}

dybit_status dybit_quantize_conv2d_requant(const dybit_conv_desc *d, const float *X, dybit_fmt fx, const float *scale_x,
                                           float *scale_x_out, void *X_packed, const void *W, dybit_fmt fw,
                                           const float *scale_w, int64_t ldw_bytes, dybit_fmt fq, const float *scale_q,
                                           const float *bias, int relu, void *Q, void *ws, size_t ws_bytes, void *stream) {
    if (d == nullptr || scale_x_out == nullptr || X_packed == nullptr) return DYBIT_ERR_INVALID_ARG;
    const dybit::QuantInput xq = {X, scale_x};
    const dybit::RequantSpec rq = {fq, scale_q, bias, relu ? 1 : 0, Q, (int64_t)d->k * fq.bits / 8};
    return dybit::conv_impl(d, X_packed, fx, scale_x_out, W, fw, scale_w, ldw_bytes, nullptr, nullptr, &rq, ws, ws_bytes,
                            stream, &xq);
}

}  // extern "C"

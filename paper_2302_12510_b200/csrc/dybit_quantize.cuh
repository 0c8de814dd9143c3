// Streaming kernels: max-abs scale, quantize + pack, decode.  All HBM-bound.
//
// Work is cut into "chunks" of 1024 consecutive codes of one row (a 1-D tensor
// is a single row).  One warp owns a chunk: eight coalesced 128-bit loads per
// lane, encode in registers, a byte-wide transpose through shared memory so
// that each lane holds 32 consecutive codes, a register bit-pack into `BITS`
// 32-bit words, and coalesced 128-bit stores.  A chunk's output always starts
// on a 16-byte boundary (1024 codes = 128 * BITS bytes).
#pragma once

#include "dybit_common.cuh"

namespace dybit {

constexpr int kChunkCodes = 1024;
constexpr int kWarpsPerBlock = 8;
constexpr int kStreamThreads = kWarpsPerBlock * 32;
constexpr int kMaxAbsmaxPartials = 1024;     // per-block maxima a max-abs launch may leave for its consumer

// ------------------------------------------------------------------ encode

// Magnitude code of a (|x| for a signed format, x itself for an unsigned one; may be negative or NaN) for M
// magnitude bits: the inverse of Eq. 1 with round-to-nearest, ties to the even code.  The result is returned with
// a bias: its low byte is the code.  `inv` is positive (or +inf when the scale underflowed).
//
// Codes grow with the value they stand for.  Below 1 they are linear, so the
// code is round(t * 2^(M-1)).  In binade e (t in [2^e, 2^(e+1)): e+1 leading
// ones, a zero, k = M-2-e fraction bits -- the encoder of Section III-B.2) the
// code is first_code(e) + round(t * 2^(k-e) - 2^k); a carry out of the
// fraction lands on the next binade's first code by itself.  Along the code
// axis these M lines (slopes 2^(M-1), 2^(M-2), 2^(M-4), ...) join up into one
// continuous concave function of t, which is therefore the smallest of them
// at every t, and it ends at the all-ones code.  Each line is ONE FMA: the
// product is a power-of-two scaling (exact), and the addend is 1.5 * 2^23 plus
// the integer constant of the line (first_code(e) - 2^k = 2^M - 3 * 2^k), so
// the FMA's single rounding is round-to-nearest-even on the final code itself
// and leaves 0x4B400000 + code in the result's bit pattern; rounding is
// monotonic, so the smallest rounded line is the rounded smallest line.
//
// Up to four magnitude bits every line is evaluated and the minimum taken
// together with the all-ones code (which also catches t beyond the top value,
// infinite included: positive floats order like their bit patterns).  Wider
// formats evaluate two lines only: the sub-unit one and the line of t's own
// binade, its constants taken straight from the exponent field of t.
template <int M>
__device__ __forceinline__ unsigned magnitude_code_biased(float a, float inv) {
    constexpr float kMagic = 12582912.0f;                                  // 1.5 * 2^23: ulp 1 on both sides
    constexpr unsigned kMagicBits = 0x4B400000u;
    // a negative product (unsigned format) and NaN (NaN input, or 0 * inf) both become 0, the code of a zero element
    const float t0 = fmaxf(__fmul_rn(a, inv), 0.0f);
    if constexpr (M <= 4) {
        unsigned best = __float_as_uint(__fmaf_rn(t0, (float)(1u << (M - 1)), kMagic));
#pragma unroll
        for (int e = 0; e + 2 <= M; ++e) {
            const int k = M - 2 - e;
            const float slope = k >= e ? (float)(1u << (k - e)) : 1.0f / (float)(1u << (e - k));
            const float addend = kMagic + (float)((1 << M) - 3 * (1 << k));
            best = min(best, __float_as_uint(__fmaf_rn(t0, slope, addend)));
        }
        return min(best, kMagicBits + ((1u << M) - 1u));
    } else {
        // largest float below the top value 2^(M-1): everything from 1.5 * 2^(M-2) up rounds to all-ones anyway
        const float below_top = __uint_as_float(((unsigned)(127 + M - 1) << 23) - 1u);
        const float t = fminf(t0, below_top);
        const unsigned sub = __float_as_uint(__fmaf_rn(t, (float)(1u << (M - 1)), kMagic));
        // exponent field of max(t, 1): the sub-unit range is folded onto binade 0
        const unsigned eb = __float_as_uint(fmaxf(t, 1.0f)) & 0x7f800000u;
        const float scale_e = __uint_as_float(((unsigned)(379 + M) << 23) - 2u * eb);                 // 2^(k-e)
        const float three_2k = __uint_as_float((((unsigned)(253 + M) << 23) | 0x400000u) - eb);       // 3 * 2^k
        const float addend = (kMagic + (float)(1u << M)) - three_2k;                                   // exact integer
        const unsigned cand = __float_as_uint(__fmaf_rn(t, scale_e, addend));
        return min(sub, cand);
    }
}

// Four elements -> four codes, one per byte of the result.
template <int BITS, bool SIGNED>
__device__ __forceinline__ unsigned encode4(const float4 v, const float inv) {
    constexpr int M = SIGNED ? BITS - 1 : BITS;
    if constexpr (SIGNED) {
        const unsigned m0 = magnitude_code_biased<M>(fabsf(v.x), inv);
        const unsigned m1 = magnitude_code_biased<M>(fabsf(v.y), inv);
        const unsigned m2 = magnitude_code_biased<M>(fabsf(v.z), inv);
        const unsigned m3 = magnitude_code_biased<M>(fabsf(v.w), inv);
        const unsigned mags = __byte_perm(__byte_perm(m0, m1, 0x0040), __byte_perm(m2, m3, 0x0040), 0x5410);
        // top byte of each float carries its sign in bit 7
        const unsigned tops = __byte_perm(__byte_perm(__float_as_uint(v.x), __float_as_uint(v.y), 0x0073),
                                          __byte_perm(__float_as_uint(v.z), __float_as_uint(v.w), 0x0073), 0x5410);
        // bit 7 of each byte set where the magnitude code is non-zero (codes are < 128)
        const unsigned nonzero = (mags + 0x7f7f7f7fu) | mags;
        return mags | (((tops & nonzero) >> (7 - M)) & (0x01010101u << M));
    } else {
        // no sign bit: negative inputs (and NaN) take the nearest value the format has, 0
        const unsigned m0 = magnitude_code_biased<M>(v.x, inv);
        const unsigned m1 = magnitude_code_biased<M>(v.y, inv);
        const unsigned m2 = magnitude_code_biased<M>(v.z, inv);
        const unsigned m3 = magnitude_code_biased<M>(v.w, inv);
        return __byte_perm(__byte_perm(m0, m1, 0x0040), __byte_perm(m2, m3, 0x0040), 0x5410);
    }
}

// ------------------------------------------------------------------ absmax

__device__ __forceinline__ unsigned finite_abs_bits(float v) {
    unsigned b = __float_as_uint(v) & 0x7fffffffu;
    return b < 0x7f800000u ? b : 0u;
}

// One thread's share of a flat run of n floats (thread tid of nthreads): scalar head up to the first 16-byte
// boundary, vector body, scalar tail.  Returns the largest finite |x| it saw, as raw bits.
template <bool STREAM>   // STREAM: evict-first loads (tensor larger than L2); otherwise leave it in L2 for the next pass
__device__ __forceinline__ unsigned absmax_flat_share(const float *__restrict__ x, int64_t n, int64_t tid, int64_t nthreads) {
    unsigned best = 0;
    int64_t head = ((16 - (reinterpret_cast<uintptr_t>(x) & 15)) & 15) / 4;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / 4;
    const float4 *xv = reinterpret_cast<const float4 *>(x + head);
    // sixteen independent 16-byte loads per thread and round trip (the ragged end reads zeros instead): with
    // three blocks per SM one round covers 29 MB, so the activations of a ResNet layer take a single round
    constexpr int kUnroll = 16;
    for (int64_t i = tid; i < nvec; i += kUnroll * nthreads) {
        float4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t iu = i + u * nthreads;
            v[u] = iu < nvec ? (STREAM ? __ldcs(xv + iu) : __ldg(xv + iu)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            best = max(best, max(max(finite_abs_bits(v[u].x), finite_abs_bits(v[u].y)),
                                 max(finite_abs_bits(v[u].z), finite_abs_bits(v[u].w))));
        }
    }
    if (tid < head) best = max(best, finite_abs_bits(x[tid]));
    const int64_t tail0 = head + nvec * 4;
    if (tail0 + tid < n) best = max(best, finite_abs_bits(x[tail0 + tid]));   // tail < 4 elements
    return best;
}

// Block-wide maximum; the result is valid in thread 0.
__device__ __forceinline__ unsigned block_max_bits(unsigned best) {
    best = __reduce_max_sync(0xffffffffu, best);
    __shared__ unsigned warp_best[kWarpsPerBlock];
    if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
    __syncthreads();
    unsigned b = 0;
    if (threadIdx.x < 32) {
        b = threadIdx.x < kWarpsPerBlock ? warp_best[threadIdx.x] : 0u;
        b = __reduce_max_sync(0xffffffffu, b);
    }
    return b;
}

// Largest finite |x| as raw fp32 bits (non-negative floats order like their
// bit patterns), max-reduced into slot[0]; slot[1] counts finished blocks.  The
// host zeroes both words beforehand.  The block that finishes last turns the
// pair into {scale, 1/scale} for m magnitude bits: amax / 2^(m-1) and one IEEE
// division 2^(m-1) / amax ({1, 1} for an all-zero tensor).
// Handles rows x cols with leading dimension ld (ld == cols: one flat run).
// With `partials` set the kernel stops one step earlier: block b stores its own maximum in partials[b] (no
// atomics, no ticket, nothing to zero beforehand) and the consumer folds the gridDim.x words itself
// (scale_from_partials); `slot` is then unused.
template <bool STREAM>
__global__ void __launch_bounds__(kStreamThreads, 3)
absmax_kernel(const float *__restrict__ x, int64_t rows, int64_t cols, int64_t ld,
              unsigned *__restrict__ slot, int m, unsigned *__restrict__ partials) {
    unsigned best = 0;
    pdl_enter();
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    if (ld == cols) {
        best = absmax_flat_share<STREAM>(x, rows * cols, tid, nthreads);
    } else {
        const int64_t total = rows * cols;
        for (int64_t i = tid; i < total; i += nthreads) {
            const int64_t r = i / cols, c = i - r * cols;
            best = max(best, finite_abs_bits(x[r * ld + c]));
        }
    }
    const unsigned b = block_max_bits(best);
    if (threadIdx.x == 0 && partials != nullptr) {
        if (DYBIT_CHECK(blockIdx.x < (unsigned)kMaxAbsmaxPartials, 0x20)) partials[blockIdx.x] = b;
    } else if (threadIdx.x == 0) {
        if (b != 0u) atomicMax(slot, b);                 // result unused: a fire-and-forget reduction
        __threadfence();
        const unsigned ticket = atomicAdd(slot + 1, 1u);
        if (ticket == gridDim.x - 1) {
            __threadfence();
            const float amax = __uint_as_float(atomicMax(slot, 0u));     // the final maximum, read at L2
            float *scale = reinterpret_cast<float *>(slot);
            if (amax == 0.0f) {
                scale[0] = 1.0f;
                scale[1] = 1.0f;
            } else {
                const float vmax = (float)(1u << (m - 1));
                scale[0] = __fdiv_rn(amax, vmax);
                scale[1] = __fdiv_rn(vmax, amax);
            }
        }
    }
}

// The partials mode of absmax_kernel for several tensors in ONE launch: blocks [first_block[l], first_block[l + 1])
// belong to tensor l and leave their maxima in partials[l][0 .. blocks of l).
constexpr int kMaxGroupLayers = 32;
struct AbsmaxLayers {
    int n_layers;
    int first_block[kMaxGroupLayers + 1];
    const float *x[kMaxGroupLayers];
    long long n[kMaxGroupLayers];
    unsigned *partials[kMaxGroupLayers];
};

__global__ void __launch_bounds__(kStreamThreads, 3) absmax_layers_kernel(const __grid_constant__ AbsmaxLayers g) {
    pdl_enter();
    int l = 0;
    while (l + 1 < g.n_layers && (int)blockIdx.x >= g.first_block[l + 1]) ++l;
    const int bid = (int)blockIdx.x - g.first_block[l], nblk = g.first_block[l + 1] - g.first_block[l];
    const unsigned best = absmax_flat_share<false>(g.x[l], (int64_t)g.n[l], (int64_t)bid * blockDim.x + threadIdx.x,
                                                   (int64_t)nblk * blockDim.x);
    const unsigned b = block_max_bits(best);
    if (threadIdx.x == 0 && DYBIT_CHECK(bid < kMaxAbsmaxPartials, 0x26)) g.partials[l][bid] = b;
}

// Consumer side of the partials mode of absmax_kernel: every block folds the per-block maxima (written by the
// previous kernel of the stream) into the tensor's maximum and derives the same {scale, 1/scale} pair with the
// same two IEEE operations as the ticket path; the block called with `writer` also stores the pair for later kernels.  Returns 1/scale.
// Must be called by all threads of the block, after pdl_enter().
__device__ __forceinline__ float scale_from_partials(const unsigned *__restrict__ partials, int n_partials, int m,
                                                     float *__restrict__ scale_out, bool writer) {
    __shared__ unsigned s_part[kWarpsPerBlock];
    __shared__ float s_inv;
    unsigned b = 0;
    for (int i = threadIdx.x; i < n_partials; i += blockDim.x) b = max(b, __ldcg(partials + i));
    b = __reduce_max_sync(0xffffffffu, b);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = b;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) b = max(b, s_part[w]);
        const float amax = __uint_as_float(b);
        float sc = 1.0f, inv = 1.0f;
        if (amax != 0.0f) {
            const float vmax = (float)(1u << (m - 1));
            sc = __fdiv_rn(amax, vmax);
            inv = __fdiv_rn(vmax, amax);
        }
        s_inv = inv;
        if (writer) {
            scale_out[0] = sc;
            scale_out[1] = inv;
        }
    }
    __syncthreads();
    return s_inv;
}

// Empty tensor: no reduction runs, the scale is {1, 1}.
__global__ void unit_scale_kernel(float *scale) {
    pdl_enter();
    scale[0] = 1.0f;
    scale[1] = 1.0f;
}

// ------------------------------------------------------------------ quantize + pack

// Packs this lane's 32 consecutive codes (bytes, low to high) into BITS words.
template <int BITS>
__device__ __forceinline__ void pack32(const unsigned (&cw)[8], unsigned (&out)[BITS]) {
    if constexpr (BITS == 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = cw[i];
        return;
    } else if constexpr (BITS == 4) {
        // bytes {a,b,c,d} -> (a | b<<4) in byte 0 and (c | d<<4) in byte 2, then gather the even bytes
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const unsigned lo = cw[2 * i] | (cw[2 * i] >> 4), hi = cw[2 * i + 1] | (cw[2 * i + 1] >> 4);
            out[i] = __byte_perm(lo, hi, 0x6420);
        }
        return;
    } else if constexpr (BITS == 2) {
        unsigned b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const unsigned t = cw[i] | (cw[i] >> 6);       // byte 0: a | b<<2, byte 2: c | d<<2
            b[i] = t | (t >> 12);                           // byte 0: a | b<<2 | c<<4 | d<<6
        }
        out[0] = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
        out[1] = __byte_perm(__byte_perm(b[4], b[5], 0x0040), __byte_perm(b[6], b[7], 0x0040), 0x5410);
        return;
    }
    // other widths: the four codes of a word shrink to 4 * BITS bits in two steps (pairs inside each 16-bit half,
    // then the halves), and the eight pieces are laid end to end; every shift is a compile-time constant
    constexpr unsigned kPair = (1u << (2 * BITS)) - 1u;
    unsigned q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const unsigned u = (cw[i] & 0x00ff00ffu) | ((cw[i] >> (8 - BITS)) & ((((1u << BITS) - 1u) << BITS) * 0x00010001u));
        q[i] = (u & kPair) | ((u >> (16 - 2 * BITS)) & (kPair << (2 * BITS)));
    }
#pragma unroll
    for (int i = 0; i < BITS; ++i) out[i] = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int pos = i * 4 * BITS, word = pos >> 5, off = pos & 31;
        out[word] |= q[i] << off;
        if (off + 4 * BITS > 32) out[word + 1] |= q[i] >> (32 - off);
    }
}

template <int BITS, bool SIGNED>
__global__ void __launch_bounds__(kStreamThreads, 3)
quantize_pack_kernel(const float *__restrict__ x, int64_t rows, int64_t cols, int64_t ld,
                     const float *__restrict__ scale, uint8_t *__restrict__ out,
                     int64_t row_stride_bytes, int64_t chunks_per_row) {
    __shared__ __align__(16) unsigned s_codes[kWarpsPerBlock][kChunkCodes / 4];
    __shared__ __align__(16) unsigned s_words[kWarpsPerBlock][32 * BITS];

    pdl_enter();
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const float inv = __ldg(scale + 1);
    const int64_t items = rows * chunks_per_row;
    const int64_t warp0 = (int64_t)blockIdx.x * kWarpsPerBlock + warp;
    const int64_t nwarps = (int64_t)gridDim.x * kWarpsPerBlock;
    constexpr int kChunkBytes = kChunkCodes * BITS / 8;       // 128 * BITS
    constexpr int kChunkVecs = kChunkBytes / 16;              // 8 * BITS

    for (int64_t item = warp0; item < items; item += nwarps) {
        const int64_t row = item / chunks_per_row;
        const int64_t chunk = item - row * chunks_per_row;
        const int64_t c0 = chunk * kChunkCodes;
        const float *src = x + row * ld + c0;
        const int64_t valid = min((int64_t)kChunkCodes, max((int64_t)0, cols - c0));
        const int64_t bytes_left = row_stride_bytes - chunk * kChunkBytes;
        const int nvec = (int)min((int64_t)kChunkVecs, bytes_left / 16);
        const bool vec_ok = (reinterpret_cast<uintptr_t>(src) & 15) == 0;

        float4 v[8];
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
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            s_codes[warp][j * 32 + lane] = encode4<BITS, SIGNED>(v[j], inv);
        }
        __syncwarp();
        // lane takes codes [32*lane, 32*lane + 32); the two 16-byte halves are
        // read in lane-dependent order so that a quarter-warp spreads over all banks
        unsigned cw[8];
        {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(&s_codes[warp][lane * 8]);
            const int first = (lane >> 2) & 1;
            uint4 a = s4[first], b = s4[first ^ 1];
            if (first) { uint4 t = a; a = b; b = t; }
            cw[0] = a.x; cw[1] = a.y; cw[2] = a.z; cw[3] = a.w;
            cw[4] = b.x; cw[5] = b.y; cw[6] = b.z; cw[7] = b.w;
        }
        unsigned w[BITS];
        pack32<BITS>(cw, w);
        uint8_t *dst = out + row * row_stride_bytes + chunk * kChunkBytes;
        if (!DYBIT_CHECK(row < rows && chunk * kChunkBytes + (int64_t)nvec * 16 <= row_stride_bytes, 0x21)) continue;
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

// ------------------------------------------------------------------ decode

struct FloatTable { float v[256]; };

// Inverse of pack32: BITS words -> this lane's 32 codes as bytes in 8 words.  Every shift is a compile-time
// constant: the eight 4 * BITS-bit pieces are cut out of the words, each is spread over two 16-bit halves and each
// half over two bytes.
template <int BITS>
__device__ __forceinline__ void unpack32(const unsigned (&in)[BITS], unsigned (&cw)[8]) {
    if constexpr (BITS == 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) cw[i] = in[i];
        return;
    } else if constexpr (BITS == 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const unsigned lo = in[i] & 0x0f0f0f0fu, hi = (in[i] >> 4) & 0x0f0f0f0fu;      // even / odd codes
            cw[2 * i] = __byte_perm(lo, hi, 0x5140);
            cw[2 * i + 1] = __byte_perm(lo, hi, 0x7362);
        }
        return;
    }
    constexpr unsigned kPiece = (BITS == 8) ? 0xffffffffu : ((1u << (4 * BITS % 32)) - 1u);
    constexpr unsigned kPair = (1u << (2 * BITS)) - 1u;
    constexpr unsigned kCode = (1u << BITS) - 1u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int pos = i * 4 * BITS, word = pos >> 5, off = pos & 31;
        unsigned q = in[word] >> off;
        if (off + 4 * BITS > 32) q |= in[word + 1] << (32 - off);
        q &= kPiece;
        const unsigned u = (q & kPair) | ((q << (16 - 2 * BITS)) & (kPair << 16));
        cw[i] = (u & (kCode * 0x00010001u)) | ((u << (8 - BITS)) & ((kCode << 8) * 0x00010001u));
    }
}

template <int BITS>
__global__ void __launch_bounds__(kStreamThreads)
decode_kernel(const uint8_t *__restrict__ packed, int64_t n, const float *__restrict__ scale,
              const __grid_constant__ FloatTable table, float *__restrict__ out) {
    __shared__ float s_lut[256];
    __shared__ __align__(16) unsigned s_words[kWarpsPerBlock][32 * BITS];
    __shared__ __align__(16) unsigned s_codes[kWarpsPerBlock][kChunkCodes / 4];
    pdl_enter();
    const float sc = scale ? __ldg(scale) : 1.0f;
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = __fmul_rn(sc, table.v[i]);
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    constexpr int kChunkBytes = kChunkCodes * BITS / 8;
    constexpr int kChunkVecs = kChunkBytes / 16;
    const int64_t packed_bytes = ((n * BITS + 7) / 8 + 15) / 16 * 16;
    const int64_t items = (n + kChunkCodes - 1) / kChunkCodes;
    const int64_t warp0 = (int64_t)blockIdx.x * kWarpsPerBlock + warp;
    const int64_t nwarps = (int64_t)gridDim.x * kWarpsPerBlock;
    const bool out_vec_ok = (reinterpret_cast<uintptr_t>(out) & 15) == 0;

    for (int64_t item = warp0; item < items; item += nwarps) {
        const int64_t c0 = item * kChunkCodes;
        const int64_t valid = min((int64_t)kChunkCodes, n - c0);
        const int nvec = (int)min((int64_t)kChunkVecs, (packed_bytes - item * kChunkBytes) / 16);
        const uint4 *src = reinterpret_cast<const uint4 *>(packed + item * kChunkBytes);
        uint4 *s4 = reinterpret_cast<uint4 *>(&s_words[warp][0]);
        for (int i = lane; i < kChunkVecs; i += 32) s4[i] = (i < nvec) ? __ldcs(src + i) : make_uint4(0, 0, 0, 0);
        __syncwarp();
        unsigned w[BITS], cw[8];
#pragma unroll
        for (int i = 0; i < BITS; ++i) w[i] = s_words[warp][lane * BITS + i];
        unpack32<BITS>(w, cw);
        {
            uint4 *c4 = reinterpret_cast<uint4 *>(&s_codes[warp][lane * 8]);
            c4[0] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
            c4[1] = make_uint4(cw[4], cw[5], cw[6], cw[7]);
        }
        __syncwarp();
        float *dst = out + c0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const unsigned c = s_codes[warp][j * 32 + lane];
            float4 r;
            r.x = s_lut[c & 0xffu];
            r.y = s_lut[(c >> 8) & 0xffu];
            r.z = s_lut[(c >> 16) & 0xffu];
            r.w = s_lut[c >> 24];
            const int64_t i0 = j * 128 + lane * 4;
            if (!DYBIT_CHECK(c0 + i0 < n || i0 >= valid, 0x22)) continue;
            if (out_vec_ok && i0 + 3 < valid) {
                __stcs(reinterpret_cast<float4 *>(dst + i0), r);
            } else {
                if (i0 + 0 < valid) dst[i0 + 0] = r.x;
                if (i0 + 1 < valid) dst[i0 + 1] = r.y;
                if (i0 + 2 < valid) dst[i0 + 2] = r.z;
                if (i0 + 3 < valid) dst[i0 + 3] = r.w;
            }
        }
        __syncwarp();
    }
}

// ------------------------------------------------------------------ RMSE (Eq. 2)

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Squared error of one element, added to s.  Only the magnitude code is needed: a signed format is symmetric, so
// |x| is compared with the magnitude's value; an unsigned one sends negative inputs to code 0.  lut[m] is the
// fp32 product scale * value(m), widened to double once per block.
template <int BITS, bool SIGNED>
__device__ __forceinline__ double sq_err_acc(float v, double dv, const double *__restrict__ lut, float inv, double s) {
    constexpr int M = SIGNED ? BITS - 1 : BITS;
    const float a = SIGNED ? fabsf(v) : fmaxf(v, 0.0f);
    const unsigned m = magnitude_code_biased<M>(a, inv) & 0xffu;
    const double e = (SIGNED ? fabs(dv) : dv) - lut[m];
    return fma(e, e, s);
}

// One pass over x: sum of d, d^2 (d = x - x[0], a shift that keeps the variance well conditioned and makes it
// exactly 0 for a constant tensor) and of e^2, e = x - xhat with xhat the fp32 quantize-dequantize image.
// acc[0..2] collect the three sums (zero on entry), acc[3] (as an integer) counts finished blocks; the last
// block replaces them by {RMSE, sigma, mse, n}.
template <int BITS, bool SIGNED>
__global__ void __launch_bounds__(kStreamThreads)
rmse_kernel(const float *__restrict__ x, int64_t n, const float *__restrict__ scale, const __grid_constant__ FloatTable table,
            double *__restrict__ acc) {
    __shared__ double s_lut[256];
    __shared__ double s_part[kWarpsPerBlock][3];
    pdl_enter();
    const float sc = __ldg(scale), inv = __ldg(scale + 1);
    // the first 2^M entries of either kind of table are the magnitudes
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = (double)__fmul_rn(sc, fabsf(table.v[i]));
    __syncthreads();
    const double shift = (double)__ldg(x);
    double sd = 0.0, sd2 = 0.0, se2 = 0.0;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    int64_t head = ((16 - (reinterpret_cast<uintptr_t>(x) & 15)) & 15) / 4;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / 4;
    const float4 *xv = reinterpret_cast<const float4 *>(x + head);
    auto one = [&](float v) {
        const double dv = (double)v;
        const double d = dv - shift;
        sd += d;
        sd2 = fma(d, d, sd2);
        se2 = sq_err_acc<BITS, SIGNED>(v, dv, s_lut, inv, se2);
    };
    constexpr int kUnroll = 4;                        // loads in flight per thread
    int64_t i = tid;
    for (; i + (kUnroll - 1) * nthreads < nvec; i += kUnroll * nthreads) {
        float4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = __ldcs(xv + i + u * nthreads);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            one(v[u].x);
            one(v[u].y);
            one(v[u].z);
            one(v[u].w);
        }
    }
    for (; i < nvec; i += nthreads) {
        const float4 v = __ldcs(xv + i);
        one(v.x);
        one(v.y);
        one(v.z);
        one(v.w);
    }
    const int64_t tail0 = head + nvec * 4;
    for (int64_t k = tid; k < head + (n - tail0); k += nthreads) one(x[k < head ? k : tail0 + (k - head)]);
    sd = warp_sum(sd);
    sd2 = warp_sum(sd2);
    se2 = warp_sum(se2);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        s_part[warp][0] = sd;
        s_part[warp][1] = sd2;
        s_part[warp][2] = se2;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0, c = 0.0;
        for (int w = 0; w < kWarpsPerBlock; ++w) {
            a += s_part[w][0];
            b += s_part[w][1];
            c += s_part[w][2];
        }
        atomicAdd(acc + 0, a);
        atomicAdd(acc + 1, b);
        atomicAdd(acc + 2, c);
        __threadfence();
        unsigned long long *ticket = reinterpret_cast<unsigned long long *>(acc + 3);
        if (atomicAdd(ticket, 1ull) == (unsigned long long)gridDim.x - 1ull) {
            __threadfence();
            const double sum_d = atomicAdd(acc + 0, 0.0), sum_d2 = atomicAdd(acc + 1, 0.0), sum_e2 = atomicAdd(acc + 2, 0.0);
            const double dn = (double)n;
            double var = (sum_d2 - sum_d * sum_d / dn) / dn;
            if (var < 0.0) var = 0.0;
            const double sigma = sqrt(var), mse = sum_e2 / dn;
            acc[0] = sigma > 0.0 ? sqrt(mse) / sigma : 0.0;
            acc[1] = sigma;
            acc[2] = mse;
            acc[3] = dn;
        }
    }
}

template <int BITS>
static dybit_status launch_rmse_bits(const float *x, int64_t n, bool is_signed, const float *scale, const FloatTable &t,
                                     double *out, cudaStream_t s) {
    int64_t blocks = (n / 4 + kStreamThreads * 4 - 1) / (kStreamThreads * 4);
    const int64_t cap = (int64_t)sm_count() * 4;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (is_signed) launch_k(rmse_kernel<BITS, true>, dim3((unsigned)blocks), dim3(kStreamThreads), 0, s, x, n, scale, t, out);
    else launch_k(rmse_kernel<BITS, false>, dim3((unsigned)blocks), dim3(kStreamThreads), 0, s, x, n, scale, t, out);
    return launch_status();
}

// ------------------------------------------------------------------ RMSE of several candidates in one pass

constexpr int kSweepMaxCand = 16;
constexpr int kSweepUnroll = 4;

// Candidate formats and the magnitude tables they decode with: the table for m magnitude bits (2^m floats)
// starts at mags[2^m - 2]; a signed code carries its sign in bit m.
struct SweepParams {
    int n_cand;
    unsigned char bits[kSweepMaxCand];
    unsigned char sgn[kSweepMaxCand];
    float mags[512];
};

// Sum of squared errors of U float4 groups (and their widened copies) under one candidate.
template <int BITS, bool SIGNED, int U>
__device__ __forceinline__ double sweep_sq_err(const float4 (&v)[U], const double (&dv)[U][4], const double *__restrict__ lut,
                                               float inv) {
    double s = 0.0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        s = sq_err_acc<BITS, SIGNED>(v[u].x, dv[u][0], lut, inv, s);
        s = sq_err_acc<BITS, SIGNED>(v[u].y, dv[u][1], lut, inv, s);
        s = sq_err_acc<BITS, SIGNED>(v[u].z, dv[u][2], lut, inv, s);
        s = sq_err_acc<BITS, SIGNED>(v[u].w, dv[u][3], lut, inv, s);
    }
    return s;
}

template <int U>
__device__ __forceinline__ double sweep_dispatch(int bits, int sgn, const float4 (&v)[U], const double (&dv)[U][4],
                                                 const double *lut, float inv) {
    switch (bits * 2 + sgn) {
        case 4: return sweep_sq_err<2, false, U>(v, dv, lut, inv);
        case 5: return sweep_sq_err<2, true, U>(v, dv, lut, inv);
        case 6: return sweep_sq_err<3, false, U>(v, dv, lut, inv);
        case 7: return sweep_sq_err<3, true, U>(v, dv, lut, inv);
        case 8: return sweep_sq_err<4, false, U>(v, dv, lut, inv);
        case 9: return sweep_sq_err<4, true, U>(v, dv, lut, inv);
        case 10: return sweep_sq_err<5, false, U>(v, dv, lut, inv);
        case 11: return sweep_sq_err<5, true, U>(v, dv, lut, inv);
        case 12: return sweep_sq_err<6, false, U>(v, dv, lut, inv);
        case 13: return sweep_sq_err<6, true, U>(v, dv, lut, inv);
        case 14: return sweep_sq_err<7, false, U>(v, dv, lut, inv);
        case 15: return sweep_sq_err<7, true, U>(v, dv, lut, inv);
        case 16: return sweep_sq_err<8, false, U>(v, dv, lut, inv);
        default: return sweep_sq_err<8, true, U>(v, dv, lut, inv);
    }
}

// One pass over x for n_cand candidate (format, scale) pairs: x is read once, every candidate's squared error is
// accumulated per thread in shared memory.  acc holds 4 doubles per candidate, zero on entry; while the kernel
// runs acc[0], acc[1] collect the sums of d and d^2 (d = x - x[0]), acc[4c + 2] candidate c's squared error and
// acc[3] (as an integer) the finished blocks.  The last block replaces them by {RMSE, sigma, mse, n} per
// candidate and writes the index of the smallest RMSE (lowest index among equals) to *best if that is given.
// Dynamic shared memory: n_cand * (256 + blockDim) doubles.
__global__ void __launch_bounds__(kStreamThreads)
rmse_sweep_kernel(const float *__restrict__ x, int64_t n, const float *__restrict__ scales,
                  const __grid_constant__ SweepParams sp, double *__restrict__ acc, int *__restrict__ best) {
    extern __shared__ __align__(16) unsigned char sweep_smem[];
    double *s_acc = reinterpret_cast<double *>(sweep_smem);                                  // [n_cand][blockDim]
    double *s_lut = s_acc + (size_t)sp.n_cand * kStreamThreads;                              // [n_cand][256] magnitudes
    __shared__ double s_part[kWarpsPerBlock][2];
    __shared__ float s_inv[kSweepMaxCand];
    pdl_enter();
    const int nc = sp.n_cand;
    for (int i = threadIdx.x; i < nc * 256; i += blockDim.x) {
        const int c = i >> 8, code = i & 255;
        const int m = sp.bits[c] - sp.sgn[c];
        s_lut[i] = code < (1 << m) ? (double)__fmul_rn(__ldg(scales + 2 * c), sp.mags[(1 << m) - 2 + code]) : 0.0;
    }
    for (int c = 0; c < nc; ++c) s_acc[c * kStreamThreads + threadIdx.x] = 0.0;
    if (threadIdx.x < nc) s_inv[threadIdx.x] = __ldg(scales + 2 * threadIdx.x + 1);
    __syncthreads();
    const double shift = (double)__ldg(x);
    double sd = 0.0, sd2 = 0.0;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    int64_t head = ((16 - (reinterpret_cast<uintptr_t>(x) & 15)) & 15) / 4;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / 4;
    const float4 *xv = reinterpret_cast<const float4 *>(x + head);
    auto moments = [&](float v) {
        const double dv = (double)v;
        const double d = dv - shift;
        sd += d;
        sd2 = fma(d, d, sd2);
        return dv;
    };
    int64_t i = tid;
    for (; i + (kSweepUnroll - 1) * nthreads < nvec; i += kSweepUnroll * nthreads) {
        float4 v[kSweepUnroll];
#pragma unroll
        for (int u = 0; u < kSweepUnroll; ++u) v[u] = __ldcs(xv + i + u * nthreads);
        double dv[kSweepUnroll][4];
#pragma unroll
        for (int u = 0; u < kSweepUnroll; ++u) {
            dv[u][0] = moments(v[u].x);
            dv[u][1] = moments(v[u].y);
            dv[u][2] = moments(v[u].z);
            dv[u][3] = moments(v[u].w);
        }
#pragma unroll 1
        for (int c = 0; c < nc; ++c)
            s_acc[c * kStreamThreads + threadIdx.x] += sweep_dispatch<kSweepUnroll>(sp.bits[c], sp.sgn[c], v, dv, s_lut + c * 256, s_inv[c]);
    }
    for (; i < nvec; i += nthreads) {
        float4 v[1] = {__ldcs(xv + i)};
        double dv[1][4];
        dv[0][0] = moments(v[0].x);
        dv[0][1] = moments(v[0].y);
        dv[0][2] = moments(v[0].z);
        dv[0][3] = moments(v[0].w);
#pragma unroll 1
        for (int c = 0; c < nc; ++c)
            s_acc[c * kStreamThreads + threadIdx.x] += sweep_dispatch<1>(sp.bits[c], sp.sgn[c], v, dv, s_lut + c * 256, s_inv[c]);
    }
    // the few elements before the first and after the last aligned group of four, one per thread
    const int64_t tail0 = head + nvec * 4;
    for (int64_t k = tid; k < head + (n - tail0); k += nthreads) {
        const float e = x[k < head ? k : tail0 + (k - head)];
        // padded with zeros, which every format represents exactly: they add no error
        float4 v[1] = {make_float4(e, 0.0f, 0.0f, 0.0f)};
        const double dv[1][4] = {{moments(e), 0.0, 0.0, 0.0}};
#pragma unroll 1
        for (int c = 0; c < nc; ++c)
            s_acc[c * kStreamThreads + threadIdx.x] += sweep_dispatch<1>(sp.bits[c], sp.sgn[c], v, dv, s_lut + c * 256, s_inv[c]);
    }
    sd = warp_sum(sd);
    sd2 = warp_sum(sd2);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        s_part[warp][0] = sd;
        s_part[warp][1] = sd2;
    }
    __syncthreads();
    // warp w adds up the candidates w, w + 8, ...
    for (int c = warp; c < nc; c += kWarpsPerBlock) {
        double t = 0.0;
        for (int k = lane; k < kStreamThreads; k += 32) t += s_acc[c * kStreamThreads + k];
        t = warp_sum(t);
        if (lane == 0) {
            atomicAdd(acc + 4 * c + 2, t);
            __threadfence();
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < kWarpsPerBlock; ++w) {
            a += s_part[w][0];
            b += s_part[w][1];
        }
        atomicAdd(acc + 0, a);
        atomicAdd(acc + 1, b);
        __threadfence();
        unsigned long long *ticket = reinterpret_cast<unsigned long long *>(acc + 3);
        if (atomicAdd(ticket, 1ull) == (unsigned long long)gridDim.x - 1ull) {
            __threadfence();
            const double sum_d = atomicAdd(acc + 0, 0.0), sum_d2 = atomicAdd(acc + 1, 0.0);
            const double dn = (double)n;
            double var = (sum_d2 - sum_d * sum_d / dn) / dn;
            if (var < 0.0) var = 0.0;
            const double sigma = sqrt(var);
            int arg = 0;
            double lowest = 0.0;
            for (int c = 0; c < nc; ++c) {
                const double mse = atomicAdd(acc + 4 * c + 2, 0.0) / dn;
                const double r = sigma > 0.0 ? sqrt(mse) / sigma : 0.0;
                acc[4 * c + 0] = r;
                acc[4 * c + 1] = sigma;
                acc[4 * c + 2] = mse;
                acc[4 * c + 3] = dn;
                if (c == 0 || r < lowest) {
                    lowest = r;
                    arg = c;
                }
            }
            if (best) *best = arg;
        }
    }
}

// ------------------------------------------------------------------ fake quantization (QAT forward / backward)

// y = scale * value(encode(x)): the quantize-dequantize image in one streaming pass, codes never stored.
// lut[m] = fmul_rn(scale, value(m)) for the magnitude codes; a signed format mirrors them.
template <int BITS, bool SIGNED>
__device__ __forceinline__ float fake_quant_one(float v, const float *__restrict__ lut, float inv) {
    constexpr int M = SIGNED ? BITS - 1 : BITS;
    // fmaxf(., 0) maps NaN to 0, as the encoder does
    const float a = SIGNED ? fmaxf(fabsf(v), 0.0f) : fmaxf(v, 0.0f);
    const unsigned m = magnitude_code_biased<M>(a, inv) & 0xffu;
    const float q = lut[m];
    // a zero magnitude carries no sign (the encoder never emits "minus zero")
    return (SIGNED && m != 0u) ? copysignf(q, v) : q;
}

template <int BITS, bool SIGNED>
__global__ void __launch_bounds__(kStreamThreads, 8)
fake_quant_kernel(const float *__restrict__ x, int64_t n, const float *__restrict__ scale,
                  const __grid_constant__ FloatTable table, float *__restrict__ y) {
    __shared__ float s_lut[256];
    pdl_enter();
    const float sc = __ldg(scale), inv = __ldg(scale + 1);
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = __fmul_rn(sc, fabsf(table.v[i]));
    __syncthreads();
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    // vector body only when x and y share their 16-byte phase
    const bool same_phase = ((reinterpret_cast<uintptr_t>(x) ^ reinterpret_cast<uintptr_t>(y)) & 15) == 0;
    int64_t head = same_phase ? ((16 - (reinterpret_cast<uintptr_t>(x) & 15)) & 15) / 4 : n;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / 4;
    const float4 *xv = reinterpret_cast<const float4 *>(x + head);
    float4 *yv = reinterpret_cast<float4 *>(y + head);
    constexpr int kUnroll = 4;
    int64_t i = tid;
    for (; i + (kUnroll - 1) * nthreads < nvec; i += kUnroll * nthreads) {
        float4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = __ldcs(xv + i + u * nthreads);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float4 r;
            r.x = fake_quant_one<BITS, SIGNED>(v[u].x, s_lut, inv);
            r.y = fake_quant_one<BITS, SIGNED>(v[u].y, s_lut, inv);
            r.z = fake_quant_one<BITS, SIGNED>(v[u].z, s_lut, inv);
            r.w = fake_quant_one<BITS, SIGNED>(v[u].w, s_lut, inv);
            __stcs(yv + i + u * nthreads, r);
        }
    }
    for (; i < nvec; i += nthreads) {
        const float4 v = __ldcs(xv + i);
        float4 r;
        r.x = fake_quant_one<BITS, SIGNED>(v.x, s_lut, inv);
        r.y = fake_quant_one<BITS, SIGNED>(v.y, s_lut, inv);
        r.z = fake_quant_one<BITS, SIGNED>(v.z, s_lut, inv);
        r.w = fake_quant_one<BITS, SIGNED>(v.w, s_lut, inv);
        __stcs(yv + i, r);
    }
    const int64_t tail0 = head + nvec * 4;
    for (int64_t k = tid; k < head + (n - tail0); k += nthreads) {
        const int64_t j = k < head ? k : tail0 + (k - head);
        y[j] = fake_quant_one<BITS, SIGNED>(x[j], s_lut, inv);
    }
}

// Straight-through backward with clipping: the gradient passes where x lies inside [lo, hi], the range the format
// covers under this scale (lo = -hi for a signed format, 0 for an unsigned one; hi = scale * 2^(m-1)), else 0.
__global__ void __launch_bounds__(kStreamThreads)
fake_quant_backward_kernel(const float *__restrict__ x, const float *__restrict__ gy, int64_t n,
                           const float *__restrict__ scale, float top, int is_signed, float *__restrict__ gx) {
    pdl_enter();
    const float hi = __fmul_rn(__ldg(scale), top), lo = is_signed ? -hi : 0.0f;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const uintptr_t px = reinterpret_cast<uintptr_t>(x), pg = reinterpret_cast<uintptr_t>(gy), po = reinterpret_cast<uintptr_t>(gx);
    const bool same_phase = (((px ^ pg) | (px ^ po)) & 15) == 0;
    int64_t head = same_phase ? ((16 - (px & 15)) & 15) / 4 : n;
    if (head > n) head = n;
    const int64_t nvec = (n - head) / 4;
    const float4 *xv = reinterpret_cast<const float4 *>(x + head);
    const float4 *gv = reinterpret_cast<const float4 *>(gy + head);
    float4 *ov = reinterpret_cast<float4 *>(gx + head);
    auto pass = [&](float v, float g) { return (v >= lo && v <= hi) ? g : 0.0f; };
    constexpr int kUnroll = 2;
    int64_t i = tid;
    for (; i + (kUnroll - 1) * nthreads < nvec; i += kUnroll * nthreads) {
        float4 v[kUnroll], g[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            v[u] = __ldcs(xv + i + u * nthreads);
            g[u] = __ldcs(gv + i + u * nthreads);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            __stcs(ov + i + u * nthreads, make_float4(pass(v[u].x, g[u].x), pass(v[u].y, g[u].y), pass(v[u].z, g[u].z), pass(v[u].w, g[u].w)));
    }
    for (; i < nvec; i += nthreads) {
        const float4 v = __ldcs(xv + i), g = __ldcs(gv + i);
        __stcs(ov + i, make_float4(pass(v.x, g.x), pass(v.y, g.y), pass(v.z, g.z), pass(v.w, g.w)));
    }
    const int64_t tail0 = head + nvec * 4;
    for (int64_t k = tid; k < head + (n - tail0); k += nthreads) {
        const int64_t j = k < head ? k : tail0 + (k - head);
        gx[j] = pass(x[j], gy[j]);
    }
}

template <int BITS>
static dybit_status launch_fake_quant_bits(const float *x, int64_t n, bool is_signed, const float *scale, const FloatTable &t,
                                           float *y, cudaStream_t s) {
    int64_t blocks = (n / 4 + kStreamThreads * 4 - 1) / (kStreamThreads * 4);
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (is_signed) launch_k(fake_quant_kernel<BITS, true>, dim3((unsigned)blocks), dim3(kStreamThreads), 0, s, x, n, scale, t, y);
    else launch_k(fake_quant_kernel<BITS, false>, dim3((unsigned)blocks), dim3(kStreamThreads), 0, s, x, n, scale, t, y);
    return launch_status();
}

// ------------------------------------------------------------------ host launchers

static int stream_grid(int64_t items_per_warp_unit) {
    // persistent-style grid: a few blocks per SM, never more than the work
    int64_t blocks = (items_per_warp_unit + kWarpsPerBlock - 1) / kWarpsPerBlock;
    int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// With `partials` (room for kMaxAbsmaxPartials words) the kernel leaves one maximum per block there and
// *n_partials says how many; the consumer finishes the reduction (scale_from_partials) and scale_out is not touched.
static dybit_status launch_absmax(const float *x, int64_t rows, int64_t cols, int64_t ld, dybit_fmt fmt,
                                  float *scale_out, cudaStream_t s, unsigned *partials = nullptr,
                                  int *n_partials = nullptr) {
    const int64_t n = rows * cols;
    if (partials == nullptr) DYBIT_CUDA_TRY(cudaMemsetAsync(scale_out, 0, 2 * sizeof(float), s));
    else if (n <= 0) return DYBIT_ERR_INVALID_ARG;
    if (n > 0) {
        // few, fat blocks: every block ends with two atomics on the same words
        int64_t blocks = (n / 4 + kStreamThreads * 16 - 1) / (kStreamThreads * 16);
        int64_t cap = (int64_t)sm_count() * 3;          // what the register file holds at once
        if (cap > kMaxAbsmaxPartials) cap = kMaxAbsmaxPartials;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        if (n_partials) *n_partials = (int)blocks;
        if (n * 4 > ((int64_t)64 << 20))
            launch_k(absmax_kernel<true>, dim3((unsigned)((int)blocks)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, x, rows, cols, ld,
                                                                       reinterpret_cast<unsigned *>(scale_out), mag_bits(fmt), partials);
        else
            launch_k(absmax_kernel<false>, dim3((unsigned)((int)blocks)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, x, rows, cols, ld,
                                                                        reinterpret_cast<unsigned *>(scale_out), mag_bits(fmt), partials);
        return launch_status();
    }
    launch_k(unit_scale_kernel, dim3((unsigned)(1)), dim3((unsigned)(1)), (size_t)(0), s, scale_out);
    return launch_status();
}

template <int BITS>
static dybit_status launch_quantize_bits(const float *x, int64_t rows, int64_t cols, int64_t ld, bool is_signed,
                                         const float *scale, uint8_t *out, int64_t row_stride_bytes,
                                         cudaStream_t s) {
    constexpr int kChunkBytes = kChunkCodes * BITS / 8;
    const int64_t chunks_per_row = (row_stride_bytes + kChunkBytes - 1) / kChunkBytes;
    const int64_t items = rows * chunks_per_row;
    if (items == 0) return DYBIT_OK;
    const int grid = stream_grid(items);
    if (is_signed)
        launch_k(quantize_pack_kernel<BITS, true>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, x, rows, cols, ld, scale, out,
                                                                        row_stride_bytes, chunks_per_row);
    else
        launch_k(quantize_pack_kernel<BITS, false>, dim3((unsigned)(grid)), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, x, rows, cols, ld, scale, out,
                                                                         row_stride_bytes, chunks_per_row);
    return launch_status();
}

static dybit_status launch_quantize(const float *x, int64_t rows, int64_t cols, int64_t ld, dybit_fmt fmt,
                                    const float *scale, uint8_t *out, int64_t row_stride_bytes,
                                    cudaStream_t s) {
    const bool sg = fmt.is_signed != 0;
    switch (fmt.bits) {
        case 2: return launch_quantize_bits<2>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
        case 3: return launch_quantize_bits<3>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
        case 4: return launch_quantize_bits<4>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
        case 5: return launch_quantize_bits<5>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
        case 6: return launch_quantize_bits<6>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
        case 7: return launch_quantize_bits<7>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
        case 8: return launch_quantize_bits<8>(x, rows, cols, ld, sg, scale, out, row_stride_bytes, s);
    }
    return DYBIT_ERR_INVALID_ARG;
}

template <int BITS>
static dybit_status launch_decode_bits(const uint8_t *packed, int64_t n, const float *scale,
                                       const FloatTable &table, float *out, cudaStream_t s) {
    const int64_t items = (n + kChunkCodes - 1) / kChunkCodes;
    if (items == 0) return DYBIT_OK;
    launch_k(decode_kernel<BITS>, dim3((unsigned)(stream_grid(items))), dim3((unsigned)(kStreamThreads)), (size_t)(0), s, packed, n, scale, table, out);
    return launch_status();
}

}  // namespace dybit

extern "C" {

dybit_status dybit_absmax_scale(const float *x, int64_t n, dybit_fmt fmt, float *scale_out, void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || n < 0 || scale_out == nullptr || (n > 0 && x == nullptr)) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(scale_out, 4)) return DYBIT_ERR_ALIGNMENT;
    return launch_absmax(x, 1, n, n, fmt, scale_out, static_cast<cudaStream_t>(stream));
}

dybit_status dybit_quantize_pack(const float *x, int64_t n, dybit_fmt fmt, const float *scale, void *packed,
                                 float *scale_out, void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || n < 0) return DYBIT_ERR_INVALID_ARG;
    if (n > 0 && (x == nullptr || packed == nullptr)) return DYBIT_ERR_INVALID_ARG;
    if (scale == nullptr && scale_out == nullptr) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(packed, 16) || !aligned(scale, 4) || !aligned(scale_out, 4))
        return DYBIT_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (scale == nullptr) {
        dybit_status st = launch_absmax(x, 1, n, n, fmt, scale_out, s);
        if (st != DYBIT_OK) return st;
        scale = scale_out;
    } else if (scale_out != nullptr && scale_out != scale) {
        DYBIT_CUDA_TRY(cudaMemcpyAsync(scale_out, scale, 2 * sizeof(float), cudaMemcpyDeviceToDevice, s));
    }
    if (n == 0) return DYBIT_OK;
    return launch_quantize(x, 1, n, n, fmt, scale, static_cast<uint8_t *>(packed),
                           (int64_t)dybit_packed_bytes(n, fmt.bits), s);
}

dybit_status dybit_quantize_pack_2d(const float *x, int64_t rows, int64_t cols, int64_t ld, dybit_fmt fmt,
                                    const float *scale, void *packed, int64_t row_stride_bytes,
                                    float *scale_out, void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || rows < 0 || cols <= 0 || ld < cols) return DYBIT_ERR_INVALID_ARG;
    if (rows > 0 && (x == nullptr || packed == nullptr)) return DYBIT_ERR_INVALID_ARG;
    if (scale == nullptr && scale_out == nullptr) return DYBIT_ERR_INVALID_ARG;
    if (row_stride_bytes < (int64_t)dybit_row_stride_bytes(cols, fmt.bits)) return DYBIT_ERR_INVALID_ARG;
    if (row_stride_bytes % 16 != 0 || !aligned(x, 4) || !aligned(packed, 16) || !aligned(scale, 4) ||
        !aligned(scale_out, 4))
        return DYBIT_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (scale == nullptr) {
        dybit_status st = launch_absmax(x, rows, cols, ld, fmt, scale_out, s);
        if (st != DYBIT_OK) return st;
        scale = scale_out;
    } else if (scale_out != nullptr && scale_out != scale) {
        DYBIT_CUDA_TRY(cudaMemcpyAsync(scale_out, scale, 2 * sizeof(float), cudaMemcpyDeviceToDevice, s));
    }
    if (rows == 0) return DYBIT_OK;
    return launch_quantize(x, rows, cols, ld, fmt, scale, static_cast<uint8_t *>(packed), row_stride_bytes, s);
}

dybit_status dybit_decode(const void *packed, int64_t n, dybit_fmt fmt, const float *scale, float *out,
                          void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || n < 0) return DYBIT_ERR_INVALID_ARG;
    if (n > 0 && (packed == nullptr || out == nullptr)) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(packed, 16) || !aligned(out, 4) || !aligned(scale, 4)) return DYBIT_ERR_ALIGNMENT;
    if (n == 0) return DYBIT_OK;
    FloatTable table;
    fill_table(fmt, table.v);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint8_t *p = static_cast<const uint8_t *>(packed);
    switch (fmt.bits) {
        case 2: return launch_decode_bits<2>(p, n, scale, table, out, s);
        case 3: return launch_decode_bits<3>(p, n, scale, table, out, s);
        case 4: return launch_decode_bits<4>(p, n, scale, table, out, s);
        case 5: return launch_decode_bits<5>(p, n, scale, table, out, s);
        case 6: return launch_decode_bits<6>(p, n, scale, table, out, s);
        case 7: return launch_decode_bits<7>(p, n, scale, table, out, s);
        case 8: return launch_decode_bits<8>(p, n, scale, table, out, s);
    }
    return DYBIT_ERR_INVALID_ARG;
}

dybit_status dybit_rmse(const float *x, int64_t n, dybit_fmt fmt, const float *scale, double *out, void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || n < 0 || out == nullptr || scale == nullptr || (n > 0 && x == nullptr)) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(out, 8) || !aligned(scale, 4)) return DYBIT_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DYBIT_CUDA_TRY(cudaMemsetAsync(out, 0, 4 * sizeof(double), s));
    if (n == 0) return DYBIT_OK;                      // {0, 0, 0, 0}
    FloatTable table;
    fill_table(fmt, table.v);
    const bool sg = fmt.is_signed != 0;
    switch (fmt.bits) {
        case 2: return launch_rmse_bits<2>(x, n, sg, scale, table, out, s);
        case 3: return launch_rmse_bits<3>(x, n, sg, scale, table, out, s);
        case 4: return launch_rmse_bits<4>(x, n, sg, scale, table, out, s);
        case 5: return launch_rmse_bits<5>(x, n, sg, scale, table, out, s);
        case 6: return launch_rmse_bits<6>(x, n, sg, scale, table, out, s);
        case 7: return launch_rmse_bits<7>(x, n, sg, scale, table, out, s);
        case 8: return launch_rmse_bits<8>(x, n, sg, scale, table, out, s);
    }
    return DYBIT_ERR_INVALID_ARG;
}

dybit_status dybit_rmse_sweep(const float *x, int64_t n, int n_cand, const dybit_fmt *fmts, const float *scales,
                              double *out, int *best, void *stream) {
    using namespace dybit;
    if (n_cand < 1 || n_cand > kSweepMaxCand || fmts == nullptr || n < 0 || out == nullptr || scales == nullptr ||
        (n > 0 && x == nullptr))
        return DYBIT_ERR_INVALID_ARG;
    for (int c = 0; c < n_cand; ++c)
        if (!fmt_ok(fmts[c])) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(out, 8) || !aligned(scales, 4) || !aligned(best, 4)) return DYBIT_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DYBIT_CUDA_TRY(cudaMemsetAsync(out, 0, (size_t)n_cand * 4 * sizeof(double), s));
    if (best) DYBIT_CUDA_TRY(cudaMemsetAsync(best, 0, sizeof(int), s));
    if (n == 0) return DYBIT_OK;
    SweepParams sp = {};
    sp.n_cand = n_cand;
    for (int c = 0; c < n_cand; ++c) {
        sp.bits[c] = (unsigned char)fmts[c].bits;
        sp.sgn[c] = fmts[c].is_signed ? 1 : 0;
    }
    // magnitude tables: m = 1..7 are the non-negative half of the signed (m+1)-bit format, m = 8 is unsigned 8-bit
    float full[256];
    for (int m = 1; m <= 8; ++m) {
        const dybit_fmt f = {m == 8 ? 8 : m + 1, m == 8 ? 0 : 1};
        fill_table(f, full);
        for (int k = 0; k < (1 << m); ++k) sp.mags[(1 << m) - 2 + k] = full[k];
    }
    const size_t smem = (size_t)n_cand * (256 + kStreamThreads) * sizeof(double);
    static std::atomic<bool> configured[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(rmse_sweep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            kSweepMaxCand * (256 + kStreamThreads) * 8));
        configured[dev] = true;
    }
    int64_t blocks = (n / 4 + kStreamThreads * kSweepUnroll - 1) / (kStreamThreads * kSweepUnroll);
    const int64_t cap = (int64_t)sm_count() * 4;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    launch_k(rmse_sweep_kernel, dim3((unsigned)blocks), dim3(kStreamThreads), smem, s, x, n, scales, sp, out, best);
    return launch_status();
}

dybit_status dybit_fake_quant(const float *x, int64_t n, dybit_fmt fmt, const float *scale, float *y, void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || n < 0 || scale == nullptr || (n > 0 && (x == nullptr || y == nullptr))) return DYBIT_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(y, 4) || !aligned(scale, 4)) return DYBIT_ERR_ALIGNMENT;
    if (n == 0) return DYBIT_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    FloatTable table;
    fill_table(fmt, table.v);
    const bool sg = fmt.is_signed != 0;
    switch (fmt.bits) {
        case 2: return launch_fake_quant_bits<2>(x, n, sg, scale, table, y, s);
        case 3: return launch_fake_quant_bits<3>(x, n, sg, scale, table, y, s);
        case 4: return launch_fake_quant_bits<4>(x, n, sg, scale, table, y, s);
        case 5: return launch_fake_quant_bits<5>(x, n, sg, scale, table, y, s);
        case 6: return launch_fake_quant_bits<6>(x, n, sg, scale, table, y, s);
        case 7: return launch_fake_quant_bits<7>(x, n, sg, scale, table, y, s);
        case 8: return launch_fake_quant_bits<8>(x, n, sg, scale, table, y, s);
    }
    return DYBIT_ERR_INVALID_ARG;
}

dybit_status dybit_fake_quant_backward(const float *x, const float *gy, int64_t n, dybit_fmt fmt, const float *scale,
                                       float *gx, void *stream) {
    using namespace dybit;
    if (!fmt_ok(fmt) || n < 0 || scale == nullptr || (n > 0 && (x == nullptr || gy == nullptr || gx == nullptr)))
        return DYBIT_ERR_INVALID_ARG;
    if (!aligned(x, 4) || !aligned(gy, 4) || !aligned(gx, 4) || !aligned(scale, 4)) return DYBIT_ERR_ALIGNMENT;
    if (n == 0) return DYBIT_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int64_t blocks = (n / 4 + kStreamThreads * 2 - 1) / (kStreamThreads * 2);
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const float top = ldexpf(1.0f, fmt.bits - (fmt.is_signed ? 1 : 0) - 1);      // Eq. 1: the largest value is 2^(m-1)
    launch_k(fake_quant_backward_kernel, dim3((unsigned)blocks), dim3(kStreamThreads), 0, s, x, gy, n, scale, top,
             fmt.is_signed ? 1 : 0, gx);
    return launch_status();
}

}  // extern "C"



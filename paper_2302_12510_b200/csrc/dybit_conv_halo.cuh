// Stride-1 convolution as an implicit GEMM whose A tile is a halo tile kept in shared memory.
//
// The im2col lowering of dybit_gemm_kernel fetches every input pixel once per filter tap (R*S times), and for
// layers with few output channels the rate at which the TMA unit fills shared-memory rows, not the tensor
// pipe, sets the pace.  Here an output tile is a rectangle of `th` rows x 8 columns of output pixels (of `ni`
// consecutive images when the feature map is small), and for each filter column s and each channel block ONE
// tiled TMA load brings the (th + R - 1) x 8 input pixels that the R taps (r, s) of that rectangle need:
// every pixel is fetched S times instead of R*S times.  Row m = 8*g + w of the MMA's A operand is output pixel
// (row g, column w) of the rectangle; its tap (r, s) is pixel row g + r of the copy for column s, i.e. the same
// shared-memory tile read from a start address r*8 pixel rows further on.  8 pixel rows are one swizzle
// pattern (8 x SWB bytes), so every start address stays aligned to the pattern and the descriptors are the
// ordinary K-major ones.
//
// Shared-memory layout of one A stage: [image j][pixel row][8 columns][SWB bytes], image j starting at
// 8 * j * hb rows (hb = th + R - 1); 16 + R - 1 pixel rows in all, of which the last few may be stale when
// ni * hb is smaller: they only feed accumulator rows that are never stored.
//
// Warp roles as in dybit_gemm_kernel: warp 0 = TMA producer (A ring and B ring have barriers of their own),
// warp 1 = tcgen05.mma issuer (accumulators double-buffered in TMEM), warps 2-9 = epilogue (fp32 through 4-D TMA
// stores that clip the rectangle to the image, the raw int32 sums, or the re-quantizing epilogue).
#pragma once

#include "dybit_gemm.cuh"

namespace dybit {

using namespace sm100;

constexpr int kHaloMaxR = 4;                          // filter rows the A stage is sized for
constexpr int kHaloRows = (16 + kHaloMaxR - 1) * 8;   // pixel rows x 8 columns = shared-memory rows of one A stage
constexpr int kHaloMaxA = 8, kHaloMaxB = 18;          // ring depths the barrier block is sized for (B: slots)
constexpr int kHaloMaxG = 8;                          // B slots are released in groups of R (one per A stage)
constexpr int kHaloCStage = kBM * 128;
constexpr int kHaloSmemBudget = 227 * 1024;

struct HaloParams {
    GemmParams g;            // output, scales, epilogue options; M = n * OH * OW, N = output channels
    int n_img;
    int th, hb, ni;          // output rows per image in a tile, th + R - 1, images per tile
    int trows, tcols;        // tiles per image column / row
    int cbs;                 // SWB-byte channel blocks per pixel
    int pad_h, pad_w;        // window origin of output pixel (oh, ow): input row oh - pad_h, column ow - pad_w
    int force;               // 1: the caller's workspace layout admits no other lowering (space-to-depth stem)
    int na, nb;              // ring depths: A stages; B slots = whole groups of R (one group per A stage)
    int b_res;               // 1: the whole weight panel (R*S*cbs blocks) is loaded once per CTA
    int m_tiles, n_tiles;
};

__device__ __forceinline__ void tma_load_4d(void *smem_dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                            uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3),
        "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, const void *smem_src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(smem_src))
                 : "memory");
}

struct HaloTile { int n_blk, img0, oh0, ow0; };

__device__ __forceinline__ HaloTile halo_tile(const HaloParams &hp, int tile) {
    HaloTile t;
    t.n_blk = tile % hp.n_tiles;
    int mt = tile / hp.n_tiles;
    t.ow0 = (mt % hp.tcols) * 8;
    mt /= hp.tcols;
    t.oh0 = (mt % hp.trows) * hp.th;
    t.img0 = (mt / hp.trows) * hp.ni;
    return t;
}

// Output row (pixel index in NHW order) of accumulator row rt of a tile, or -1 when that row is not an output.
__device__ __forceinline__ int halo_row(const HaloParams &hp, const HaloTile &t, int rt) {
    const int g = rt >> 3, w = rt & 7;
    const int j = g / hp.hb, hl = g - j * hp.hb;
    const int img = t.img0 + j, oh = t.oh0 + hl, ow = t.ow0 + w;
    if (j >= hp.ni || hl >= hp.th || img >= hp.n_img || oh >= hp.g.OH || ow >= hp.g.OW) return -1;
    return (img * hp.g.OH + oh) * hp.g.OW + ow;
}

// Narrow tiles on 64-byte pixels (BN = 64, SWB = 64) leave the tensor pipe idle between their short MMAs while one
// thread walks through waits and commits; two CTAs per SM (each takes 128 TMEM columns and under half of the shared
// memory when the weight panel is resident) fill each other's gaps.
template <int BN, int SWB>
constexpr int halo_ctas_per_sm() { return (BN == 64 && SWB == 64) ? 2 : 1; }

// CTA `bid` of the `nblk` CTAs that work on the layer (tensor maps and parameters live in the kernel's parameter
// space, whichever kernel below passes them).
template <Kind KIND, int BN, int SWB>
__device__ __forceinline__ void conv_halo_body(const CUtensorMap &tmap_x, const CUtensorMap &tmap_w, const CUtensorMap &tmap_y,
                                               const HaloParams &hp, const int bid, const int nblk) {
    constexpr int kAStage = kHaloRows * SWB;
    constexpr int kBStage = BN * SWB;
    const GemmParams &p = hp.g;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *c_stages = smem;                                        // two output staging buffers (1024-byte aligned)
    uint8_t *b_stages = c_stages + 2 * kHaloCStage;                  // multiples of 4096 bytes
    uint8_t *a_stages = b_stages + (hp.b_res ? p.R * p.S * hp.cbs : hp.nb) * kBStage;   // multiples of 8 * SWB bytes
    uint64_t *bars = reinterpret_cast<uint64_t *>(a_stages + hp.na * kAStage);
    uint64_t *a_full = bars;
    uint64_t *a_empty = a_full + kHaloMaxA;
    uint64_t *b_full = a_empty + kHaloMaxA;
    uint64_t *b_gempty = b_full + kHaloMaxB;                         // one per group of R slots
    uint64_t *acc_full = b_gempty + kHaloMaxG;
    uint64_t *acc_empty = acc_full + 2;
    uint64_t *panel_full = acc_empty + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(panel_full + 1);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = hp.m_tiles * hp.n_tiles;
    constexpr uint32_t kTmemCols = 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kHaloMaxA; ++s) {
            mbar_init(&a_full[s], 1);
            mbar_init(&a_empty[s], 1);
        }
        for (int s = 0; s < kHaloMaxB; ++s) mbar_init(&b_full[s], 1);
        for (int s = 0; s < kHaloMaxG; ++s) mbar_init(&b_gempty[s], 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], kEpilogueWarps);
        }
        mbar_init(panel_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_w);
        if (p.tma_store) prefetch_tensormap(&tmap_y);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_enter();
    if (p.clock != nullptr && threadIdx.x == 32) atomicMin(p.clock, (unsigned long long)global_timer_ns());

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int sa = 0, gb = 0;                       // ring positions and the parity of the phase they wait for
            uint32_t pa = 1, pb = 1;
            const int ngroups = hp.b_res ? 1 : hp.nb / p.R;
            bool ok = true;
            const uint32_t a_bytes = (uint32_t)(hp.ni * hp.hb * 8 * SWB);
            if (hp.b_res && bid < total_tiles) {
                const int blocks = p.R * p.S * hp.cbs;
                mbar_arrive_expect_tx(panel_full, (uint32_t)blocks * kBStage);
                for (int j = 0; j < blocks; ++j) tma_load_2d(b_stages + j * kBStage, &tmap_w, j * SWB, 0, panel_full);
            }
            for (int tile = bid; tile < total_tiles && ok; tile += nblk) {
                const HaloTile t = halo_tile(hp, tile);
                for (int cb = 0; cb < hp.cbs && ok; ++cb) {
                    for (int fs = 0; fs < p.S && ok; ++fs) {
                        if (!wait_bounded(&a_empty[sa], pa, abort_flag, 1)) { ok = false; break; }
                        mbar_arrive_expect_tx(&a_full[sa], a_bytes);
                        tma_load_4d(a_stages + sa * kAStage, &tmap_x, cb * SWB, t.ow0 - hp.pad_w + fs, t.oh0 - hp.pad_h, t.img0,
                                    &a_full[sa]);
                        if (++sa == hp.na) { sa = 0; pa ^= 1u; }
                        if (hp.b_res) continue;
                        // the R weight blocks of this filter column: one group of slots, released together
                        if (!wait_bounded(&b_gempty[gb], pb, abort_flag, 7)) { ok = false; break; }
                        int kx = (fs * hp.cbs + cb) * SWB;                 // K offset of tap (0, fs), channel block cb
                        for (int fr = 0; fr < p.R; ++fr, kx += p.S * hp.cbs * SWB) {
                            const int sb = gb * p.R + fr;
                            mbar_arrive_expect_tx(&b_full[sb], kBStage);
                            tma_load_2d(b_stages + sb * kBStage, &tmap_w, kx, t.n_blk * BN, &b_full[sb]);
                        }
                        if (++gb == ngroups) { gb = 0; pb ^= 1u; }
                    }
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);      // copies in flight get a bounded time to land
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t kCFormat = (KIND == Kind::I8) ? 2u : 1u;
            constexpr uint32_t kABFormat = (KIND == Kind::F8F6F4) ? 0u : 1u;
            constexpr uint32_t idesc = umma_idesc(kCFormat, kABFormat, kBM, BN);
            // This thread runs at roughly six clocks per instruction while an MMA of a narrow tile takes under 100,
            // and a barrier probed right after a tcgen05.commit does not answer until the MMAs in flight have drained
            // (about 200 clocks; about 45 when probed between two MMAs).  So: ring positions, barrier addresses and
            // descriptor low words are running 32-bit values; every barrier is probed one step AHEAD, right after the
            // first MMA of the step before it; commits come once per A stage (the R weight slots of a filter column are
            // released together); and a wait that runs out does not branch out of the loops: it raises the abort flag,
            // after which every later wait of the CTA gives up at once and the remaining MMAs run on stale data into an
            // accumulator that the epilogue no longer stores.
            constexpr uint32_t kHi = umma_desc_hi<SWB>();
            constexpr uint32_t kA16 = kAStage >> 4, kB16 = kBStage >> 4, kTap16 = (8 * SWB) >> 4;
            const uint32_t a_lo0 = umma_desc_lo(smem_u32(a_stages)), b_lo0 = umma_desc_lo(smem_u32(b_stages));
            const uint32_t a_full0 = smem_u32(a_full), a_empty0 = smem_u32(a_empty);
            const uint32_t b_full0 = smem_u32(b_full), b_gempty0 = smem_u32(b_gempty);
            const uint32_t acc_full0 = smem_u32(acc_full), acc_empty0 = smem_u32(acc_empty);
            const uint32_t panel_step = (uint32_t)(p.S * hp.cbs) * kB16;      // resident panel: from tap (fr, fs) to (fr + 1, fs)
            const int na = hp.na, R = p.R, S = p.S, cbs = hp.cbs;
            const bool b_res = hp.b_res != 0;
            const int nslots = b_res ? 0 : hp.nb;
            int sa = 0, sb = 0;                                   // A stage, B slot
            uint32_t pa = 0, pb = 0, lt = 0;
            uint32_t a_bar = a_full0, a_lo_s = a_lo0, b_bar = b_full0, b_lo_s = b_lo0, g_bar = b_gempty0;
            bool a_ready = false, b_ready = false, acc_ready = false;
            if (b_res && bid < total_tiles) (void)wait_bounded(panel_full, 0u, abort_flag, 6);
            for (int tile = bid; tile < total_tiles; tile += nblk, ++lt) {
                const uint32_t as = lt & 1u;
                if (!acc_ready) (void)wait_bounded_addr(acc_empty0 + as * 8, ((lt >> 1) & 1u) ^ 1u, abort_flag, 2);
                acc_ready = false;
                tc_fence_after_sync();
                const uint32_t d = tmem_base + as * BN;
                uint32_t accumulate = 0;
                for (int cb = 0; cb < cbs; ++cb) {
                    for (int fs = 0; fs < S; ++fs) {
                        if (!a_ready) (void)wait_bounded_addr(a_bar, pa, abort_flag, 3);
                        tc_fence_after_sync();
                        // where the next A stage lives
                        int sa_n = sa + 1;
                        uint32_t a_bar_n = a_bar + 8, a_lo_n = a_lo_s + kA16, pa_n = pa;
                        if (sa_n == na) { sa_n = 0; a_bar_n = a_full0; a_lo_n = a_lo0; pa_n ^= 1u; }
                        uint32_t a_lo = a_lo_s;                                     // tap (0, fs); + kTap16 per filter row
                        uint32_t b_lo = b_lo0 + (uint32_t)(fs * cbs + cb) * kB16;   // (resident panel)
                        for (int fr = 0; fr < R; ++fr) {
                            if (!b_res) {
                                if (!b_ready) (void)wait_bounded_addr(b_bar, pb, abort_flag, 8);
                                tc_fence_after_sync();
                                b_lo = b_lo_s;
                            }
                            umma_lo<KIND>(d, a_lo, b_lo, kHi, idesc, accumulate);
                            accumulate = 1;
                            // look one step ahead while that MMA runs
                            if (!b_res) {
                                if (++sb == nslots) { sb = 0; b_bar = b_full0; b_lo_s = b_lo0; pb ^= 1u; }
                                else { b_bar += 8; b_lo_s += kB16; }
                                b_ready = mbar_try_wait_addr(b_bar, pb);
                            }
                            if (fr == 0) {
                                a_ready = mbar_try_wait_addr(a_bar_n, pa_n);
                                acc_ready = mbar_try_wait_addr(acc_empty0 + (as ^ 1u) * 8, (((lt + 1) >> 1) & 1u) ^ 1u);
                            }
#pragma unroll
                            for (int k = 1; k < SWB / kUmmaKBytes; ++k)
                                umma_lo<KIND>(d, a_lo + k * (kUmmaKBytes >> 4), b_lo + k * (kUmmaKBytes >> 4), kHi, idesc, 1u);
                            a_lo += kTap16;
                            b_lo += panel_step;
                        }
                        umma_commit_addr(a_empty0 + sa * 8);
                        if (!b_res) {
                            umma_commit_addr(g_bar);
                            g_bar = sb == 0 ? b_gempty0 : g_bar + 8;
                        }
                        sa = sa_n;
                        a_bar = a_bar_n;
                        a_lo_s = a_lo_n;
                        pa = pa_n;
                    }
                }
                umma_commit_addr(acc_full0 + as * 8);
            }
        }
    } else {
        // ------------------------------------------------ epilogue
        const int q = warp & 3;
        const int row_in_tile = q * 32 + lane;
        const int group = (warp - 2) >> 2;
        const bool issuer = (threadIdx.x & 127) == 64;
        const float alpha = (float)((double)__ldg(p.scale_a) * (double)__ldg(p.scale_b) * p.pow2);
        const float inv_q = p.Q ? __ldg(p.scale_q + 1) : 1.0f;
        uint32_t lt = 0;
        for (int tile = bid; tile < total_tiles; tile += nblk, ++lt) {
            const HaloTile t = halo_tile(hp, tile);
            const uint32_t as = lt & 1u, aph = (lt >> 1) & 1u;
            // one thread per group polls the accumulator's barrier; the other 127 sleep in the hardware barrier that
            // hands them the outcome (256 polling threads would keep the shared-memory pipe busy that the MMA
            // thread's own barrier probes and the arrivals of TMA and tcgen05.commit go through)
            const bool ok = named_barrier_and(1 + group, 128, issuer ? wait_bounded(&acc_full[as], aph, abort_flag, 4) : true);
            if (!ok) break;
            tc_fence_after_sync();
            const int row = halo_row(hp, t, row_in_tile);
            const uint32_t taddr = tmem_base + as * BN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int cc = group; cc < BN / 32; cc += kEpilogueWarps / 4) {
                const int col0 = t.n_blk * BN + cc * 32;
                if (col0 >= p.N) break;
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
                    if (row >= 0) {
                        if (p.bias) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < p.N) f[j] = __fadd_rn(f[j], __ldg(p.bias + col0 + j));
                        }
                        if (p.relu) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.0f);
                        }
                        requant_dispatch(p.q_bits, p.q_signed, f, inv_q,
                                         p.Q + (int64_t)row * p.ldq + (int64_t)col0 * p.q_bits / 8, p.N - col0);
                    }
                    continue;
                }
                if (KIND == Kind::I8 && p.C_raw != nullptr && row >= 0) {
                    int32_t *rrow = p.C_raw + (int64_t)row * p.ldc + col0;
                    if (col0 + 32 <= p.N && (reinterpret_cast<uintptr_t>(rrow) & 15) == 0) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            __stcs(reinterpret_cast<int4 *>(rrow) + j, make_int4((int)r[4 * j], (int)r[4 * j + 1], (int)r[4 * j + 2], (int)r[4 * j + 3]));
                    } else {
                        for (int j = 0; j < 32; ++j)
                            if (col0 + j < p.N) rrow[j] = (int)r[j];
                    }
                }
                if (!p.tma_store) {
                    // the output cannot be described to the TMA (base or rows not 16-byte aligned): each thread writes
                    // the 32 values of its own output pixel
                    if (row >= 0) {
                        float *dst = p.C + (int64_t)row * p.ldc + col0;
                        if (col0 + 32 <= p.N && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                __stcs(reinterpret_cast<float4 *>(dst) + j, make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]));
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (col0 + j < p.N) dst[j] = f[j];
                        }
                    }
                    continue;
                }
                // stage 128 rows x 32 columns in the TMA's 128-byte swizzle; one 4-D store per image of the tile writes
                // the th x 8 pixels of that image and clips what lies outside the feature map
                uint8_t *stage = c_stages + group * kHaloCStage;
                if (issuer) bulk_wait_group_read<0>();
                named_barrier(1 + group, 128);
                uint8_t *srow = stage + row_in_tile * 128;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<float4 *>(srow + ((j ^ (row_in_tile & 7)) << 4)) =
                        make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                fence_proxy_async_smem();
                named_barrier(1 + group, 128);
                if (issuer) {
                    for (int j = 0; j < hp.ni; ++j)
                        if (t.img0 + j < hp.n_img)
                            tma_store_4d(&tmap_y, stage + j * hp.hb * 1024, col0, t.ow0, t.oh0, t.img0 + j);
                    bulk_commit_group();
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[as]);
        }
        if (issuer) bulk_wait_group_read<0>();
    }

    tc_fence_before_sync();
    __syncthreads();
    if (p.clock != nullptr && threadIdx.x == 32) atomicMax(p.clock + 1, (unsigned long long)global_timer_ns());
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <Kind KIND, int BN, int SWB>
__global__ void __launch_bounds__(320, halo_ctas_per_sm<BN, SWB>())
dybit_conv_halo_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                       const __grid_constant__ CUtensorMap tmap_y, const HaloParams hp) {
    conv_halo_body<KIND, BN, SWB>(tmap_x, tmap_w, tmap_y, hp, (int)blockIdx.x, (int)gridDim.x);
}

// Several layers of one kernel configuration (and one shared-memory size) in ONE launch, as GemmMulti.
struct HaloMulti {
    int n;
    int first_block[kMaxMulti + 1];
    CUtensorMap tx[kMaxMulti], tw[kMaxMulti], ty[kMaxMulti];
    HaloParams hp[kMaxMulti];
};
static_assert(sizeof(HaloParams) <= sizeof(MultiEntry::extra), "MultiEntry::extra holds a HaloParams");

template <Kind KIND, int BN, int SWB>
__global__ void __launch_bounds__(320, halo_ctas_per_sm<BN, SWB>()) dybit_conv_halo_multi_kernel(const __grid_constant__ HaloMulti m) {
    int g = 0;
    while (g + 1 < m.n && (int)blockIdx.x >= m.first_block[g + 1]) ++g;
    conv_halo_body<KIND, BN, SWB>(m.tx[g], m.tw[g], m.ty[g], m.hp[g], (int)blockIdx.x - m.first_block[g],
                                  m.first_block[g + 1] - m.first_block[g]);
}

template <Kind KIND, int BN, int SWB>
static dybit_status launch_halo_multi(const MultiEntry *e, int n, cudaStream_t s) {
    auto kern = dybit_conv_halo_multi_kernel<KIND, BN, SWB>;
    static std::atomic<bool> configured[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kHaloSmemBudget));
        configured[dev] = true;
    }
    HaloMulti m;
    memset(&m, 0, sizeof(m));
    m.n = n;
    // (the entries of one launch share per_sm and the shared-memory size: the collector groups by both)
    multi_shares(e, n, e[0].per_sm * sm_count(), m.first_block);
    for (int i = 0; i < n; ++i) {
        m.tx[i] = e[i].ta;
        m.tw[i] = e[i].tb;
        m.ty[i] = e[i].tc;
        memcpy(&m.hp[i], e[i].extra, sizeof(HaloParams));
    }
    launch_k(kern, dim3((unsigned)m.first_block[n]), dim3(320u), (size_t)e[0].smem, s, m);
    return launch_status();
}

// ------------------------------------------------------------------ host side

// How a convolution is cut into halo tiles, or eligible = false when this lowering does not apply.
struct HaloPlan {
    bool eligible;
    int swb, cbs, th, hb, ni, trows, tcols, m_tiles;
};

// 0: by shape, 1: wherever the lowering applies, 2: never (dybit_set_conv_lowering)
static std::atomic<int> &conv_lowering_mode() {
    static std::atomic<int> mode{0};
    return mode;
}

// Tiles for a stride-1 window walk over `rows_r` filter rows: th output rows per image so that ni * (th + rows_r - 1)
// pixel rows fit the A stage.
static void halo_tiling(HaloPlan *h, int n, int oh, int ow, int rows_r) {
    const int htiles = (oh + 15) / 16;
    h->th = (oh + htiles - 1) / htiles;
    h->hb = h->th + rows_r - 1;
    h->ni = (16 + rows_r - 1) / h->hb;
    if (h->ni < 1) h->ni = 1;
    if (h->ni > n) h->ni = n;
    h->trows = htiles;
    h->tcols = (ow + 7) / 8;
    const int64_t m_tiles = (int64_t)((n + h->ni - 1) / h->ni) * h->trows * h->tcols;
    h->m_tiles = m_tiles > (1 << 24) ? 0 : (int)m_tiles;
}

static HaloPlan plan_halo(const dybit_conv_desc *d, int oh, int ow, int64_t cpb) {
    HaloPlan h = {};
    if (conv_lowering_mode().load(std::memory_order_relaxed) == 2) return h;
    const int swb = (cpb % 128 == 0) ? 128 : (cpb == 64 ? 64 : 0);
    if (swb == 0 || d->stride != 1 || d->dilation != 1 || d->r > kHaloMaxR || d->s > 16) return h;
    if (d->r == 1 && d->s == 1) return h;                       // a plain GEMM on the activation: the tiled kernel
    if (cpb / swb > 64 || d->pad > 64) return h;
    halo_tiling(&h, d->n, oh, ow, d->r);
    if (h.m_tiles == 0) return h;
    h.swb = swb;
    h.cbs = (int)(cpb / swb);
    h.eligible = true;
    return h;
}

// Expanded activation [n][h][w][cpb bytes] as a tiled 4-D map: box = swb channel bytes x 8 columns x hb rows x ni
// images; whatever lies outside the tensor (the padding ring, columns past the feature map, images past the
// batch) reads as zeros.
static dybit_status make_halo_input_map(CUtensorMap *map, const void *xe, const dybit_conv_desc *d, int64_t cpb,
                                        const HaloPlan &h) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return DYBIT_ERR_CUDA;
    cuuint64_t dims[4] = {(cuuint64_t)cpb, (cuuint64_t)d->w, (cuuint64_t)d->h, (cuuint64_t)d->n};
    cuuint64_t strides[3] = {(cuuint64_t)cpb, (cuuint64_t)cpb * d->w, (cuuint64_t)cpb * d->w * d->h};
    cuuint32_t box[4] = {(cuuint32_t)h.swb, 8, (cuuint32_t)h.hb, (cuuint32_t)h.ni};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(xe), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, h.swb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DYBIT_OK : DYBIT_ERR_CUDA;
}

// fp32 output [n][oh][ow][k] as a 4-D map whose box is 32 channels x 8 columns x th rows of one image.
static bool make_halo_output_map(CUtensorMap *map, float *Y, const dybit_conv_desc *d, int oh, int ow, const HaloPlan &h) {
    if ((reinterpret_cast<uintptr_t>(Y) & 15) != 0 || d->k % 4 != 0) return false;
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[4] = {(cuuint64_t)d->k, (cuuint64_t)ow, (cuuint64_t)oh, (cuuint64_t)d->n};
    cuuint64_t strides[3] = {(cuuint64_t)d->k * 4, (cuuint64_t)d->k * 4 * ow, (cuuint64_t)d->k * 4 * ow * oh};
    cuuint32_t box[4] = {32, 8, (cuuint32_t)h.th, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, Y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <Kind KIND, int BN, int SWB>
static dybit_status launch_halo_inst(const CUtensorMap &tx, const CUtensorMap &tw, const CUtensorMap &ty, HaloParams hp,
                                     cudaStream_t s) {
    constexpr int kAStage = kHaloRows * SWB;
    constexpr int kBStage = BN * SWB;
    const int budget = kHaloSmemBudget - 1024 - 1024 - 2 * kHaloCStage;      // alignment slack, barrier block, C staging
    const int panel = hp.g.R * hp.g.S * hp.cbs * kBStage;
    const int tiles = hp.m_tiles * hp.n_tiles;
    hp.b_res = (hp.n_tiles == 1 && tiles > sm_count() && panel + 3 * kAStage <= budget) ? 1 : 0;
    if (hp.b_res) {
        hp.na = (budget - panel) / kAStage;
        hp.nb = 0;
    } else {
        hp.na = SWB == 64 ? 4 : 3;
        int groups = (budget - hp.na * kAStage) / (kBStage * hp.g.R);       // B slots come in groups of R
        if (groups > kHaloMaxG) groups = kHaloMaxG;
        if (groups * hp.g.R > kHaloMaxB) groups = kHaloMaxB / hp.g.R;
        hp.nb = groups * hp.g.R;
    }
    if (hp.na > kHaloMaxA) hp.na = kHaloMaxA;
    // two CTAs per SM where the kernel is built for it and a resident panel leaves room: each gets half the SM
    int per_sm = 1;
    if (halo_ctas_per_sm<BN, SWB>() == 2 && hp.b_res && tiles > sm_count()) {
        const int half = 113 * 1024 - 1024 - 1024 - 2 * kHaloCStage - panel;
        if (half >= 3 * kAStage) {
            per_sm = 2;
            if (hp.na > half / kAStage) hp.na = half / kAStage;
        }
    }
    if (hp.na < 2 || (!hp.b_res && hp.nb < 2 * hp.g.R)) return DYBIT_ERR_UNSUPPORTED;
    // Measured on ResNet-18 shapes at batch 32: with two CTAs per SM and the weights resident the halo tiles beat
    // the im2col lowering (12.2 against 17.0 us on the 64 -> 64 channel 3x3 layers); with one CTA per SM and a
    // weight ring they do not (10.5 against 9.0 us at 128 channels, 15.2 against 13.0 us at 512): there the single
    // MMA-issuing thread, not the operand traffic, sets the pace, and the plainer loop of dybit_gemm_kernel wins.
    if (per_sm != 2 && !hp.force && conv_lowering_mode().load(std::memory_order_relaxed) != 1) return DYBIT_ERR_UNSUPPORTED;
    const int smem = 1024 + 2 * kHaloCStage + (hp.b_res ? panel : hp.nb * kBStage) + hp.na * kAStage + 1024;
    auto kern = dybit_conv_halo_kernel<KIND, BN, SWB>;
    static std::atomic<bool> configured[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    if (!configured[dev]) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kHaloSmemBudget));
        configured[dev] = true;
    }
    const int grid = tiles < per_sm * sm_count() ? tiles : per_sm * sm_count();
    ProfileEvents ev = profile_events();
    if constexpr (KIND == Kind::I8) {
        // inside dybit_conv2d_prepared_layers: gathered, launched together with its like at the end of that call
        // (a resident weight panel presumes CTAs that take several tiles, which a share of a launch still does)
        if (gemm_collector() != nullptr && !ev.start && !ev.stop && !ev.clock) {
            MultiEntry e;
            memset(&e, 0, sizeof(e));
            e.ta = tx;
            e.tb = tw;
            e.tc = ty;
            memcpy(e.extra, &hp, sizeof(hp));
            e.tiles = tiles;
            e.per_sm = per_sm;
            e.smem = smem;
            e.work = (double)tiles * (double)(hp.g.R * hp.g.S * hp.cbs + 8);
            gemm_collector()->add(launch_halo_multi<KIND, BN, SWB>, e);
            return DYBIT_OK;
        }
    }
    profile_events() = ProfileEvents();
    hp.g.clock = ev.clock;
    if (ev.start) DYBIT_CUDA_TRY(cudaEventRecord(ev.start, s));
    launch_k(kern, dim3((unsigned)grid), dim3(320u), (size_t)smem, s, tx, tw, ty, hp);
    const dybit_status st = launch_status();
    if (ev.stop) DYBIT_CUDA_TRY(cudaEventRecord(ev.stop, s));
    return st;
}

template <Kind KIND, int SWB>
static dybit_status launch_halo_bn(int bn, const CUtensorMap &tx, const CUtensorMap &tw, const CUtensorMap &ty,
                                   const HaloParams &hp, cudaStream_t s) {
    switch (bn) {
        case 64: return launch_halo_inst<KIND, 64, SWB>(tx, tw, ty, hp, s);
        case 128: return launch_halo_inst<KIND, 128, SWB>(tx, tw, ty, hp, s);
        default: return launch_halo_inst<KIND, 256, SWB>(tx, tw, ty, hp, s);
    }
}

template <int SWB>
static dybit_status launch_halo_kind(dybit_container cont, int bn, const CUtensorMap &tx, const CUtensorMap &tw,
                                     const CUtensorMap &ty, const HaloParams &hp, cudaStream_t s) {
    switch (cont) {
        case DYBIT_CONTAINER_I8: return launch_halo_bn<Kind::I8, SWB>(bn, tx, tw, ty, hp, s);
        case DYBIT_CONTAINER_E4M3: return launch_halo_bn<Kind::F8F6F4, SWB>(bn, tx, tw, ty, hp, s);
        default: return launch_halo_bn<Kind::F16, SWB>(bn, tx, tw, ty, hp, s);
    }
}

// Runs the convolution on the halo kernel; DYBIT_ERR_UNSUPPORTED means "use another lowering" (nothing was launched).
// xe: expanded activation [n*h*w][cpb]; we: expanded weights [k][wrb] with K order (r, s, c).
static dybit_status launch_conv_halo(dybit_container cont, const dybit_conv_desc *d, int oh, int ow, int64_t cpb,
                                     const uint8_t *xe, const uint8_t *we, int64_t wrb, const GemmParams &p_in,
                                     cudaStream_t s) {
    const HaloPlan h = plan_halo(d, oh, ow, cpb);
    if (!h.eligible) return DYBIT_ERR_UNSUPPORTED;
    HaloParams hp = {};
    hp.g = p_in;
    CUtensorMap tx, tw, ty;
    memset(&ty, 0, sizeof(ty));
    const int bn = choose_bn_tiles(h.m_tiles, d->k);
    // chosen by shape: only the configuration that runs two CTAs per SM (see launch_halo_inst); checked here as well
    // so that the other shapes do not pay for three tensor-map encodings first
    if (conv_lowering_mode().load(std::memory_order_relaxed) == 0 && !(h.swb == 64 && bn == 64 && d->k <= 64))
        return DYBIT_ERR_UNSUPPORTED;
    if (hp.g.Q == nullptr) {
        if (!make_halo_output_map(&ty, hp.g.C, d, oh, ow, h)) return DYBIT_ERR_UNSUPPORTED;
        hp.g.tma_store = 1;
    }
    dybit_status st = make_halo_input_map(&tx, xe, d, cpb, h);
    if (st != DYBIT_OK) return st;
    st = make_operand_map(&tw, we, d->k, wrb, wrb, bn, h.swb);
    if (st != DYBIT_OK) return st;
    hp.n_img = d->n;
    hp.th = h.th;
    hp.hb = h.hb;
    hp.ni = h.ni;
    hp.trows = h.trows;
    hp.tcols = h.tcols;
    hp.cbs = h.cbs;
    hp.pad_h = d->pad;
    hp.pad_w = d->pad;
    hp.m_tiles = h.m_tiles;
    hp.n_tiles = (d->k + bn - 1) / bn;
    return h.swb == 128 ? launch_halo_kind<128>(cont, bn, tx, tw, ty, hp, s) : launch_halo_kind<64>(cont, bn, tx, tw, ty, hp, s);
}

// Stride-2 convolution on at most four one-byte channels (the 3-channel 7 x 7 stem) after a 2 x 2 space-to-depth
// rearrangement of the activation (plan_conv, kConvS2D): every 2 x 2 block of input pixels is one 16-byte pixel, the
// filter becomes Rp x 4 taps walked with stride 1, and the four taps of one filter row are 64 CONTIGUOUS bytes of the
// rearranged image.  The input map therefore has rows that overlap: row w of it is the 64-byte window that starts at
// rearranged pixel w (16 bytes further on than row w - 1).  One TMA load brings the windows of th + Rp - 1 rows x 8
// columns; filter row r' is a 64-byte K block of its own, read from pixel row g + r' of that tile.  The image carries
// its horizontal padding physically (padL zero pixels in front of every row, three behind), since a window that
// starts inside the image must not be zero-filled as a whole; rows above and below the image are the TMA's zero fill.
static dybit_status launch_conv_s2d(dybit_container cont, const dybit_conv_desc *d, int oh, int ow, const S2dGeom &g,
                                    const uint8_t *xs, const uint8_t *we, int64_t wrb, const GemmParams &p_in,
                                    cudaStream_t s) {
    HaloPlan h = {};
    halo_tiling(&h, d->n, oh, ow, g.Rp);
    if (h.m_tiles == 0) return DYBIT_ERR_UNSUPPORTED;
    h.swb = 64;
    h.cbs = 1;
    HaloParams hp = {};
    hp.g = p_in;
    hp.g.R = g.Rp;
    hp.g.S = 1;
    CUtensorMap tx, tw, ty;
    memset(&ty, 0, sizeof(ty));
    hp.g.tma_store = (hp.g.Q == nullptr && make_halo_output_map(&ty, hp.g.C, d, oh, ow, h)) ? 1 : 0;
    {
        EncodeTiledFn fn = encode_tiled_fn();
        if (fn == nullptr) return DYBIT_ERR_CUDA;
        cuuint64_t dims[4] = {64, (cuuint64_t)(g.P - 3), (cuuint64_t)g.Hs, (cuuint64_t)d->n};
        cuuint64_t strides[3] = {16, (cuuint64_t)g.P * 16, (cuuint64_t)g.P * 16 * g.Hs};
        cuuint32_t box[4] = {64, 8, (cuuint32_t)h.hb, (cuuint32_t)h.ni};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (fn(&tx, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<uint8_t *>(xs), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DYBIT_ERR_CUDA;
    }
    const int bn = choose_bn_tiles(h.m_tiles, d->k);
    dybit_status st = make_operand_map(&tw, we, d->k, wrb, wrb, bn, 64);
    if (st != DYBIT_OK) return st;
    hp.n_img = d->n;
    hp.th = h.th;
    hp.hb = h.hb;
    hp.ni = h.ni;
    hp.trows = h.trows;
    hp.tcols = h.tcols;
    hp.cbs = 1;
    hp.pad_h = -g.lo_r;
    hp.pad_w = 0;                       // the left padding is in the image: window of output column ow starts at pixel ow
    hp.force = 1;
    hp.m_tiles = h.m_tiles;
    hp.n_tiles = (d->k + bn - 1) / bn;
    return launch_halo_kind<64>(cont, bn, tx, tw, ty, hp, s);
}

}  // namespace dybit

extern "C" dybit_status dybit_set_conv_lowering(int mode) {
    if (mode < 0 || mode > 2) return DYBIT_ERR_INVALID_ARG;
    dybit::conv_lowering_mode().store(mode, std::memory_order_relaxed);
    return DYBIT_OK;
}

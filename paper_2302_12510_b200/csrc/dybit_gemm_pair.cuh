// The GEMM on CTA pairs (tcgen05 cta_group::2): two neighbouring SMs share one 256 x 256 output tile.
// Each CTA loads its own 128 rows of A and HALF of the tile's 256 B rows; the tensor cores of both SMs read
// B from both shared memories, so a CTA moves 256 shared-memory rows per K block instead of the 384 that a
// 128 x 256 tile of its own needs -- the TMA unit's row rate is what bounds the single-CTA kernel.
// fp32 output through TMA stores (optionally with the raw integer sums beside it) or the re-quantizing epilogue;
// batches, convolution gathers and outputs the TMA cannot describe stay on dybit_gemm_kernel.
#pragma once

#include "dybit_gemm.cuh"

namespace dybit {

using namespace sm100;

constexpr int kPairBN = 256;                 // tile columns of the pair
constexpr int kPairStages = 6;               // 6 x (16 KB A + 16 KB half-B)
constexpr int kPairAStage = kBM * kBKBytes;
constexpr int kPairBStage = (kPairBN / 2) * kBKBytes;
constexpr int kPairCStage = kBM * 128;
constexpr int kPairSmemBytes = kPairStages * (kPairAStage + kPairBStage) + 2 * kPairCStage + 512 + 1024;

// Work items of the pair kernel.  Tiles [0, split_from) are one item each; every later tile is two items, its left and
// its right 256 x 128 half.  The host splits the tiles of a last, less than half-full wave: a half costs 0.61 of a
// whole tile (an N = 128 instruction takes 78 clocks where an N = 256 one takes 128), so the wave ends sooner.
__device__ __forceinline__ void pair_item(int item, const GemmParams &p, int &m_blk, int &n_blk, int &n_off, int &width) {
    int tile = item, half = 0;
    width = kPairBN;
    if (item >= p.split_from) {
        tile = p.split_from + ((item - p.split_from) >> 1);
        half = (item - p.split_from) & 1;
        width = kPairBN / 2;
    }
    tile_coords(tile, p.m_tiles, p.n_tiles, m_blk, n_blk);
    n_off = half * (kPairBN / 2);
}

// p.m_tiles counts 256-row blocks here; p.n_tiles counts 256-column blocks.
template <Kind KIND>
__global__ void __launch_bounds__(320, 1)
dybit_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                       const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
    constexpr int BN = kPairBN;
    constexpr int kStages = kPairStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_stages = smem;
    uint8_t *b_stages = smem + kStages * kPairAStage;
    uint8_t *c_stages = smem + kStages * (kPairAStage + kPairBStage);
    uint64_t *bars = reinterpret_cast<uint64_t *>(c_stages + 2 * kPairCStage);
    uint64_t *full = bars;                       // used in the leader CTA: both CTAs' loads complete on it
    uint64_t *empty = bars + kStages;            // one per CTA, released by the leader's multicast commit
    uint64_t *acc_full = bars + 2 * kStages;     // one per CTA, multicast commit
    uint64_t *acc_empty = acc_full + 2;          // used in the leader CTA: epilogue warps of both CTAs arrive
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();     // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;
    const int whole_tiles = p.m_tiles * p.n_tiles;
    const int total_tiles = whole_tiles + (whole_tiles - p.split_from);      // work items: a split tile counts twice
    constexpr uint32_t kTmemCols = 2 * BN;       // two accumulators of 256 columns: all of TMEM

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 2 * kEpilogueWarps);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (p.tma_store) prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                          // the peer's barriers exist before anything signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_enter();
    if (p.clock != nullptr && threadIdx.x == 32) atomicMin(p.clock, (unsigned long long)global_timer_ns());

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
                int m_blk, n_blk, n_off, width;
                pair_item(tile, p, m_blk, n_blk, n_off, width);
                const int a_row = m_blk * 2 * kBM + (int)rank * kBM;
                // (a half item still loads 128 rows of B per CTA; the instruction reads the first 64 of each)
                const int b_row = n_blk * BN + n_off + (int)rank * (width / 2);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!wait_bounded(&empty[s], ph ^ 1u, abort_flag, 1)) { ok = false; break; }
                    // the leader's barrier collects the bytes of both CTAs
                    if (rank == 0) mbar_arrive_expect_tx(&full[s], 2u * (kPairAStage + kPairBStage));
                    const uint32_t bar = mapa_u32(smem_u32(&full[s]), 0u);
                    tma_load_2d_pair(a_stages + s * kPairAStage, &tmap_a, kb * kBKBytes, a_row, bar);
                    tma_load_2d_pair(b_stages + s * kPairBStage, &tmap_b, kb * kBKBytes, b_row, bar);
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t kCFormat = (KIND == Kind::I8) ? 2u : 1u;
            constexpr uint32_t kABFormat = (KIND == Kind::F8F6F4) ? 0u : 1u;
            constexpr uint32_t idesc_whole = umma_idesc(kCFormat, kABFormat, 2 * kBM, BN);
            constexpr uint32_t idesc_half = umma_idesc(kCFormat, kABFormat, 2 * kBM, BN / 2);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs, ++lt) {
                const uint32_t idesc = tile >= p.split_from ? idesc_half : idesc_whole;
                const uint32_t as = lt & 1u, aph = (lt >> 1) & 1u;
                if (!wait_bounded(&acc_empty[as], aph ^ 1u, abort_flag, 2)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d = tmem_base + as * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1u;
                    if (!wait_bounded(&full[s], ph, abort_flag, 3)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t adesc = umma_desc_kmajor<128>(smem_u32(a_stages + s * kPairAStage));
                    const uint64_t bdesc = umma_desc_kmajor<128>(smem_u32(b_stages + s * kPairBStage));
#pragma unroll
                    for (int k = 0; k < kBKBytes / kUmmaKBytes; ++k) {
                        umma_pair<KIND>(d, adesc + (uint64_t)(k * (kUmmaKBytes >> 4)), bdesc + (uint64_t)(k * (kUmmaKBytes >> 4)),
                                        idesc, (uint32_t)((kb | k) != 0));
                    }
                    umma_commit_pair(&empty[s], (uint16_t)3);       // frees the stage in both CTAs
                }
                if (ok) umma_commit_pair(&acc_full[as], (uint16_t)3);
            }
        }
    } else {
        // ------------------------------------------------ epilogue (both CTAs): TMEM -> registers -> shared -> TMA store
        const int q = warp & 3;
        const int row_in_tile = q * 32 + lane;
        const int group = (warp - 2) >> 2;
        const bool issuer = (threadIdx.x & 127) == 64;
        const float alpha = (float)((double)__ldg(p.scale_a) * (double)__ldg(p.scale_b) * p.pow2);
        const float inv_q = p.Q ? __ldg(p.scale_q + 1) : 1.0f;
        uint32_t lt = 0;
        for (int tile = pair; tile < total_tiles; tile += num_pairs, ++lt) {
            int m_blk, n_blk, n_off, width;
            pair_item(tile, p, m_blk, n_blk, n_off, width);
            const uint32_t as = lt & 1u, aph = (lt >> 1) & 1u;
            // one outcome for the group's 128 threads, which meet in named barriers below
            const bool ok = named_barrier_and(1 + group, 128, wait_bounded(&acc_full[as], aph, abort_flag, 4));
            if (!ok) break;
            tc_fence_after_sync();
            const int row0 = m_blk * 2 * kBM + (int)rank * kBM;          // this CTA's first output row
            const uint32_t taddr = tmem_base + as * BN + ((uint32_t)(q * 32) << 16);
            const bool last_tile = tile + num_pairs >= total_tiles;
#pragma unroll 1
            for (int cc = group; cc < width / 32; cc += kEpilogueWarps / 4) {
                const int col0 = n_blk * BN + n_off + cc * 32;
                if (col0 >= p.N || row0 >= p.M) break;
                uint32_t r[32];
                tmem_ld_32x32(taddr + cc * 32, r);
                tmem_ld_wait();
                float f[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float acc = (KIND == Kind::I8) ? __int2float_rn((int)r[j]) : __uint_as_float(r[j]);
                    f[j] = __fmul_rn(acc, alpha);
                }
                const int row = row0 + row_in_tile;
                if (p.Q) {
                    // re-quantizing epilogue: + bias, ReLU, encode, pack; 32 codes of this thread's row
                    if (row < p.M) {
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
                if (KIND == Kind::I8 && p.C_raw != nullptr && row < p.M) {
                    // raw integer sums beside the fp32 result (rows are 16-byte aligned: checked on the host)
                    int32_t *rrow = p.C_raw + (int64_t)row * p.ldc + col0;
                    if (col0 + 32 <= p.N) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            __stcs(reinterpret_cast<int4 *>(rrow) + j, make_int4((int)r[4 * j], (int)r[4 * j + 1], (int)r[4 * j + 2], (int)r[4 * j + 3]));
                    } else {
                        for (int j = 0; j < 32; ++j)
                            if (col0 + j < p.N) rrow[j] = (int)r[j];
                    }
                }
                // in the CTA's last tile the operand stages are idle: every chunk takes a buffer of its own
                uint8_t *stage = last_tile ? a_stages + cc * kPairCStage : c_stages + group * kPairCStage;
                if (issuer && !last_tile) bulk_wait_group_read<0>();
                named_barrier(1 + group, 128);
                uint8_t *srow = stage + row_in_tile * 128;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<float4 *>(srow + ((j ^ (row_in_tile & 7)) << 4)) =
                        make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                fence_proxy_async_smem();
                named_barrier(1 + group, 128);
                if (issuer) {
                    tma_store_2d(&tmap_c, stage, col0, row0);
                    bulk_commit_group();
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            // the leader's MMA thread may overwrite this accumulator once all sixteen epilogue warps have let go
            if (lane == 0) mbar_arrive_cluster(mapa_u32(smem_u32(&acc_empty[as]), 0u));
        }
        if (issuer) bulk_wait_group_read<0>();
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();          // neither CTA leaves (or frees TMEM) while the other may still touch its memory
    if (p.clock != nullptr && threadIdx.x == 32) atomicMax(p.clock + 1, (unsigned long long)global_timer_ns());
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// Launches the pair kernel: clusters of two CTAs, as many as the device holds at once.
template <Kind KIND>
static dybit_status launch_gemm_pair_kind(const CUtensorMap &ta, const CUtensorMap &tb, const CUtensorMap &tc,
                                          const GemmParams &p_in, cudaStream_t s) {
    GemmParams p = p_in;
    auto kern = dybit_gemm_pair_kernel<KIND>;
    static std::atomic<int> max_clusters[64];
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(320);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    if (max_clusters[dev] == 0) {
        DYBIT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes));
        cfg.gridDim = dim3((unsigned)sm_count());
        cfg.numAttrs = 1;                      // the occupancy query wants the cluster shape only
        int n = 0;
        DYBIT_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, kern, &cfg));
        if (n < 1) return DYBIT_ERR_UNSUPPORTED;
        max_clusters[dev] = n;
    }
    const int tiles = p.m_tiles * p.n_tiles;
    const int resident = max_clusters[dev];
    const int pairs = tiles < resident ? tiles : resident;
    // a last wave that fills at most half of the pairs is worked on as halves (see pair_item)
    const int rest = tiles % pairs;
    p.split_from = (rest > 0 && 2 * rest <= pairs) ? tiles - rest : tiles;
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.numAttrs = 2;
    ProfileEvents ev = profile_events();
    profile_events() = ProfileEvents();
    p.clock = ev.clock;
    if (ev.start) DYBIT_CUDA_TRY(cudaEventRecord(ev.start, s));
    (void)cudaLaunchKernelEx(&cfg, kern, ta, tb, tc, p);
    const dybit_status st = launch_status();
    if (ev.stop) DYBIT_CUDA_TRY(cudaEventRecord(ev.stop, s));
    return st;
}

// Whether a plain GEMM goes to the pair kernel: fp32 output that the TMA can describe, nothing else asked for,
// and at least one 256 x 256 tile per pair of SMs.
static bool gemm_pair_eligible(int64_t M, int64_t N, const GemmParams &p) {
    if (p.bmt != 0) return false;
    if (p.C_raw != nullptr && ((reinterpret_cast<uintptr_t>(p.C_raw) & 15) != 0 || p.ldc % 4 != 0)) return false;
    const int64_t tiles = ((M + 255) / 256) * ((N + 255) / 256);
    return M >= 256 && N >= 256 && tiles * 2 >= sm_count();
}

static dybit_status launch_gemm_pair(dybit_container cont, const void *ae, int64_t a_row_bytes, const void *be,
                                     int64_t b_row_bytes, int64_t M, int64_t N, const GemmParams &p_in, cudaStream_t s) {
    GemmParams p = p_in;
    p.m_tiles = (int)((M + 255) / 256);
    p.n_tiles = (int)((N + kPairBN - 1) / kPairBN);
    CUtensorMap ta, tb, tc;
    // (a row of A may be shorter than a whole number of K blocks: the TMA reads zeros past its end)
    dybit_status st = make_operand_map(&ta, ae, M, a_row_bytes, a_row_bytes, kBM);
    if (st != DYBIT_OK) return st;
    st = make_operand_map(&tb, be, N, b_row_bytes, b_row_bytes, kPairBN / 2);
    if (st != DYBIT_OK) return st;
    memset(&tc, 0, sizeof(tc));
    if (p.Q == nullptr && !make_output_map(&tc, p.C, p.M, p.N, p.ldc, 0, 0)) return DYBIT_ERR_UNSUPPORTED;
    p.tma_store = p.Q == nullptr ? 1 : 0;
    switch (cont) {
        case DYBIT_CONTAINER_I8: return launch_gemm_pair_kind<Kind::I8>(ta, tb, tc, p, s);
        case DYBIT_CONTAINER_E4M3: return launch_gemm_pair_kind<Kind::F8F6F4>(ta, tb, tc, p, s);
        default: return launch_gemm_pair_kind<Kind::F16>(ta, tb, tc, p, s);
    }
}

}  // namespace dybit

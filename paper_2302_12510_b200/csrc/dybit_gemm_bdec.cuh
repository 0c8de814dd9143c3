// The GEMM with its B operand (the weights) decoded in the main loop.
//
// dybit_gemm_kernel multiplies operands that a separate launch has expanded into the container type.  Here the
// weights stay packed in global memory: the TMA brings BN rows x 64 bytes of 4-bit codes (one 128-code K block) per
// stage, four decode warps turn them into int8 through the 16-entry table held in registers (prmt lookups, the shared
// row / column decoders of Section III-B.1-2 in this machine's terms) and write them into the stage's 128-byte
// swizzled operand buffer, and tcgen05.mma consumes it.  Per weight the kernel reads 0.5 byte from global memory
// instead of 0.5 (read) + 1 (written) + 1 (read again): what pays when the weights are streamed once for few rows
// of A (M up to a few hundred), where the GEMM is bound by that stream and not by the tensor pipe.  For large
// products the expand pass stays: a 128 x 256 x 128-byte block already moves 96 KB through shared memory (TMA fill +
// operand reads) per 512 tensor-pipe clocks, and decoding in the loop adds another 48 KB per block.
//
// int8 container, B in a 4-bit format whose table the register lookup can hold (expand4_job), A expanded beforehand
// as usual; fp32 output through TMA stores, optionally the raw int32 sums.
#pragma once

#include "dybit_gemm.cuh"

namespace dybit {

using namespace sm100;

constexpr int kBdecDecodeWarps = 4;
constexpr int kBdecThreads = 32 * (2 + 4 + kBdecDecodeWarps);      // producer, MMA, 4 epilogue, 4 decode warps
constexpr int kBdecCStage = kBM * 128;

template <int BN>
struct BdecSmem {
    static constexpr int kA = kBM * kBKBytes;          // expanded A block
    static constexpr int kP = BN * (kBKBytes / 2);     // packed B block: 64 bytes per row
    static constexpr int kE = BN * kBKBytes;           // decoded B block
    static constexpr int kFit = (227 * 1024 - 2 * kBdecCStage - 1536) / (kA + kP + kE);
    static constexpr int kStages = kFit > 6 ? 6 : kFit;
    static constexpr int kBytes = kStages * (kA + kP + kE) + 2 * kBdecCStage + 512 + 1024;
};

template <int BN>
__global__ void __launch_bounds__(kBdecThreads, 1)
dybit_gemm_bdec_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_p,
                       const __grid_constant__ CUtensorMap tmap_c, const GemmParams p, const BdecTable bt) {
    using L = BdecSmem<BN>;
    constexpr int kStages = L::kStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *c_stages = smem;
    uint8_t *a_stages = c_stages + 2 * kBdecCStage;
    uint8_t *e_stages = a_stages + kStages * L::kA;
    uint8_t *p_stages = e_stages + kStages * L::kE;
    uint64_t *bars = reinterpret_cast<uint64_t *>(p_stages + kStages * L::kP);
    uint64_t *full = bars;                      // TMA: A block and packed B block have landed
    uint64_t *ready = bars + kStages;           // decode warps: the decoded B block is in place
    uint64_t *empty = bars + 2 * kStages;       // MMAs that read the stage have completed
    uint64_t *acc_full = bars + 3 * kStages;
    uint64_t *acc_empty = acc_full + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int total_tiles = p.m_tiles * p.n_tiles;
    constexpr uint32_t kTmemCols = 2 * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&ready[s], kBdecDecodeWarps);
            mbar_init(&empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 4);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_p);
        prefetch_tensormap(&tmap_c);
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
            int s = 0;
            uint32_t ph = 1;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int m_blk, n_blk;
                tile_coords(tile, p.m_tiles, p.n_tiles, m_blk, n_blk);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!wait_bounded(&empty[s], ph, abort_flag, 1)) { ok = false; break; }
                    mbar_arrive_expect_tx(&full[s], L::kA + L::kP);
                    tma_load_2d(a_stages + s * L::kA, &tmap_a, kb * kBKBytes, m_blk * kBM, &full[s]);
                    tma_load_2d(p_stages + s * L::kP, &tmap_p, kb * (kBKBytes / 2), n_blk * BN, &full[s]);
                    if (++s == kStages) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                for (int i = 0; i < 64; ++i) __nanosleep(2000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(2u, 1u, kBM, BN);
            constexpr uint32_t kHi = umma_desc_hi<128>();
            const uint32_t a_lo0 = umma_desc_lo(smem_u32(a_stages)), e_lo0 = umma_desc_lo(smem_u32(e_stages));
            const uint32_t full0 = smem_u32(full), ready0 = smem_u32(ready), empty0 = smem_u32(empty);
            int s = 0;
            uint32_t ph = 0, lt = 0;
            for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++lt) {
                const uint32_t as = lt & 1u;
                (void)wait_bounded_addr(smem_u32(&acc_empty[as]), ((lt >> 1) & 1u) ^ 1u, abort_flag, 2);
                tc_fence_after_sync();
                const uint32_t d = tmem_base + as * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    (void)wait_bounded_addr(full0 + s * 8, ph, abort_flag, 3);       // A block (TMA)
                    (void)wait_bounded_addr(ready0 + s * 8, ph, abort_flag, 9);      // B block (decode warps)
                    tc_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + s * (L::kA >> 4), e_lo = e_lo0 + s * (L::kE >> 4);
#pragma unroll
                    for (int k = 0; k < kBKBytes / kUmmaKBytes; ++k)
                        umma_lo<Kind::I8>(d, a_lo + k * (kUmmaKBytes >> 4), e_lo + k * (kUmmaKBytes >> 4), kHi, idesc,
                                          (uint32_t)((kb | k) != 0));
                    umma_commit_addr(empty0 + s * 8);
                    if (++s == kStages) { s = 0; ph ^= 1u; }
                }
                umma_commit_addr(smem_u32(&acc_full[as]));
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------ epilogue (4 warps, one TMEM lane quarter each)
        const int q = warp & 3;
        const int row_in_tile = q * 32 + lane;
        const bool issuer = warp == 2 && lane == 0;
        const float alpha = (float)((double)__ldg(p.scale_a) * (double)__ldg(p.scale_b) * p.pow2);
        uint32_t lt = 0, buf = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++lt) {
            int m_blk, n_blk;
            tile_coords(tile, p.m_tiles, p.n_tiles, m_blk, n_blk);
            const uint32_t as = lt & 1u, aph = (lt >> 1) & 1u;
            const bool ok = named_barrier_and(1, 128, issuer ? wait_bounded(&acc_full[as], aph, abort_flag, 4) : true);
            if (!ok) break;
            tc_fence_after_sync();
            const int row = m_blk * kBM + row_in_tile;
            const uint32_t taddr = tmem_base + as * BN + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int cc = 0; cc < BN / 32; ++cc) {
                const int col0 = n_blk * BN + cc * 32;
                if (col0 >= p.N) break;
                uint32_t r[32];
                tmem_ld_32x32(taddr + cc * 32, r);
                tmem_ld_wait();
                if (p.C_raw != nullptr && row < p.M) {
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
                // two staging buffers in turn: the store that last read this one (two chunks ago) must be done with it
                uint8_t *stage = c_stages + buf * kBdecCStage;
                if (issuer) bulk_wait_group_read<1>();
                named_barrier(1, 128);
                uint8_t *srow = stage + row_in_tile * 128;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float4 v;
                    v.x = __fmul_rn(__int2float_rn((int)r[4 * j]), alpha);
                    v.y = __fmul_rn(__int2float_rn((int)r[4 * j + 1]), alpha);
                    v.z = __fmul_rn(__int2float_rn((int)r[4 * j + 2]), alpha);
                    v.w = __fmul_rn(__int2float_rn((int)r[4 * j + 3]), alpha);
                    *reinterpret_cast<float4 *>(srow + ((j ^ (row_in_tile & 7)) << 4)) = v;
                }
                fence_proxy_async_smem();
                named_barrier(1, 128);
                if (issuer) {
                    tma_store_2d(&tmap_c, stage, col0, m_blk * kBM);
                    bulk_commit_group();
                }
                buf ^= 1u;
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[as]);
        }
        if (issuer) bulk_wait_group_read<0>();
    } else {
        // ------------------------------------------------ decode warps: packed 4-bit codes -> int8, swizzled operand rows
        // Four consecutive lanes share a row of 64 packed bytes (16 bytes = 32 codes each), so a quarter-warp reads 128
        // contiguous bytes; the 32 decoded bytes of a lane are chunks 2v and 2v + 1 of its row, stored at the
        // positions the 128-byte swizzle gives them (chunk c of row r lives at c ^ (r & 7)).
        const int dw = warp - 6;
        const int sub_row = lane >> 2, v = lane & 3;
        const unsigned t[4] = {bt.tab[0], bt.tab[1], bt.tab[2], bt.tab[3]};
        const bool ng = bt.neg_high != 0;
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                bool got = true;
                if (lane == 0) got = wait_bounded(&full[s], ph, abort_flag, 10);
                got = __shfl_sync(0xffffffffu, got, 0);
                if (!got) { ok = false; break; }
                const uint8_t *src = p_stages + s * L::kP;
                uint8_t *dst = e_stages + s * L::kE;
#pragma unroll 2
                for (int r0 = dw * 8; r0 < BN; r0 += kBdecDecodeWarps * 8) {
                    const int r = r0 + sub_row;
                    const uint4 w = *reinterpret_cast<const uint4 *>(src + r * (kBKBytes / 2) + v * 16);
                    uint4 o0, o1;
                    o0.x = expand4_lookup(w.x, t, ng); o0.y = expand4_lookup(w.x >> 16, t, ng);
                    o0.z = expand4_lookup(w.y, t, ng); o0.w = expand4_lookup(w.y >> 16, t, ng);
                    o1.x = expand4_lookup(w.z, t, ng); o1.y = expand4_lookup(w.z >> 16, t, ng);
                    o1.z = expand4_lookup(w.w, t, ng); o1.w = expand4_lookup(w.w >> 16, t, ng);
                    uint8_t *drow = dst + r * kBKBytes;
                    *reinterpret_cast<uint4 *>(drow + (((2 * v) ^ (r & 7)) << 4)) = o0;
                    *reinterpret_cast<uint4 *>(drow + (((2 * v + 1) ^ (r & 7)) << 4)) = o1;
                }
                fence_proxy_async_smem();                 // generic-proxy stores -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(&ready[s]);
                if (++s == kStages) { s = 0; ph ^= 1u; }
            }
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

// ------------------------------------------------------------------ host side

// 0: expand pass for both operands (default for large products); 1: decode B in the main loop wherever it applies;
// 2: by shape (few rows of A).  Set through dybit_set_gemm_decode.
static std::atomic<int> &gemm_decode_mode() {
    static std::atomic<int> mode{2};
    return mode;
}

template <int BN>
static dybit_status launch_bdec_inst(const CUtensorMap &ta, const CUtensorMap &tp, const CUtensorMap &tc, GemmParams p,
                                     const BdecTable &bt, cudaStream_t s) {
    using L = BdecSmem<BN>;
    auto kern = dybit_gemm_bdec_kernel<BN>;
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
    profile_events() = ProfileEvents();
    p.clock = ev.clock;
    if (ev.start) DYBIT_CUDA_TRY(cudaEventRecord(ev.start, s));
    launch_k(kern, dim3((unsigned)grid), dim3((unsigned)kBdecThreads), (size_t)L::kBytes, s, ta, tp, tc, p, bt);
    const dybit_status st = launch_status();
    if (ev.stop) DYBIT_CUDA_TRY(cudaEventRecord(ev.stop, s));
    return st;
}

// Whether this call can take the decode-in-the-loop kernel, by format and output alone (the mode is the caller's).
static bool gemm_bdec_applicable(dybit_container cont, dybit_fmt fb, const ElemTable &tb, const GemmParams &p, BdecTable *bt) {
    if (cont != DYBIT_CONTAINER_I8 || fb.bits != 4 || p.Q != nullptr || p.bmt != 0) return false;
    if ((reinterpret_cast<uintptr_t>(p.C) & 15) != 0 || (p.ldc * 4) % 16 != 0) return false;
    Expand4Job job;
    const ExpandOperand op = {nullptr, 4, 1, 0, 32, nullptr, 0, &tb};
    if (!expand4_job(op, 1, true, &job)) return false;
    for (int i = 0; i < 4; ++i) bt->tab[i] = job.tab[i];
    bt->neg_high = job.neg_high;
    return true;
}

// A expanded in the workspace ([M][rb] int8); B packed as the caller gave it.
static dybit_status launch_gemm_bdec(const uint8_t *ae, int64_t rb, const uint8_t *B, int64_t ldb_bytes, int64_t M, int64_t N,
                                     int64_t K, const GemmParams &p_in, const BdecTable &bt, cudaStream_t s) {
    GemmParams p = p_in;
    const int bn = choose_bn(M, N);
    CUtensorMap ta, tp, tc;
    dybit_status st = make_operand_map(&ta, ae, M, rb, rb, kBM);
    if (st != DYBIT_OK) return st;
    // packed codes: 64 bytes per 128-code K block, no swizzle (the decode warps read it with plain loads); rows past N
    // and bytes past the row's last code read as zeros = code 0 = value 0
    {
        EncodeTiledFn fn = encode_tiled_fn();
        if (fn == nullptr) return DYBIT_ERR_CUDA;
        const int64_t row_bytes = round_up(K, 128) / 2;
        cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)N};
        cuuint64_t strides[1] = {(cuuint64_t)ldb_bytes};
        cuuint32_t box[2] = {(cuuint32_t)(kBKBytes / 2), (cuuint32_t)bn};
        cuuint32_t estr[2] = {1, 1};
        if (fn(&tp, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t *>(B), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DYBIT_ERR_CUDA;
    }
    if (!make_output_map(&tc, p.C, p.M, p.N, p.ldc, 0, 0)) return DYBIT_ERR_UNSUPPORTED;
    p.tma_store = 1;
    p.k_blocks = (int)(rb / kBKBytes);
    p.m_tiles = (int)((M + kBM - 1) / kBM);
    p.n_tiles = (int)((N + bn - 1) / bn);
    switch (bn) {
        case 64: return launch_bdec_inst<64>(ta, tp, tc, p, bt, s);
        case 128: return launch_bdec_inst<128>(ta, tp, tc, p, bt, s);
        default: return launch_bdec_inst<256>(ta, tp, tc, p, bt, s);
    }
}

}  // namespace dybit

extern "C" dybit_status dybit_set_gemm_decode(int mode) {
    if (mode < 0 || mode > 2) return DYBIT_ERR_INVALID_ARG;
    dybit::gemm_decode_mode().store(mode, std::memory_order_relaxed);
    return DYBIT_OK;
}

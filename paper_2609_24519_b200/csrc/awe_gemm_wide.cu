// FP4 products with 64-bit running sums (Algorithm 1, third loop and last step) for encodings whose
// reconstruction sum does not fit 32 bits even over one 256-element K block -- the 12-product
// FP16-significand encoding (Appendix A: |2AB| <= 2 * 2047^2 * K).
//
// Same structure as the 32-bit kernel (persistent CTA pairs, TMA ring, tcgen05.mma kind::mxf4 with
// constant block scales, epilogue warps that fold l_k * P_k into register-resident sums), but a
// pair owns a 256 x 128 tile so that each epilogue thread keeps 64 columns as 64-bit integers
// (128 registers).  With 128-column accumulators two of them and the scale bytes fit tensor
// memory side by side, so the accumulators are fully independent.
#include <cstdio>
#include <cstdlib>

#include "gemm_common.cuh"

namespace awe {
using namespace gemm;
namespace {

constexpr int kN = 128;                        // tile columns
constexpr int kBRows = kN / 2;                 // rows of the B plane staged by each CTA of the pair
constexpr int kBBytes = kBRows * kBlockKBytes;  // 8 KB
constexpr int kStageBytes = kABytes + kBBytes;  // 24 KB
constexpr int kStages = 8;
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + kEpiWarps * kStageWarpBytes + 256;
constexpr uint32_t kAcc0 = 0, kAcc1 = kN;
// mxf4 instruction descriptor: E2M1 x E2M1, both K-major, UE8M0 scales, M = 256 (pair), N = 128, K = 64
constexpr uint32_t kIdesc =
    (1u << 7) | (1u << 10) | ((uint32_t)(kN >> 3) << 17) | (1u << 23) | ((uint32_t)((kTileM * 2) >> 4) << 24);

struct SharedW {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
};

__device__ __forceinline__ bool wait(SharedW* sh, uint32_t bar, uint32_t parity, unsigned int* status, int site) {
    return bounded_wait_ns(&sh->abort_flag, bar, parity, status, site, kWaitLimitNs);
}

template <int BLK>
__device__ __forceinline__ void drain_block64(uint32_t taddr, long long (&sum)[64], float acc_scale, int ell) {
    uint32_t v[32];
    ptx::tmem_ld_32x32(taddr + BLK * 32, v);
    ptx::tmem_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i)
        sum[BLK * 32 + i] += (long long)ell * (long long)__float2int_rn(__uint_as_float(v[i]) * acc_scale);
}

__global__ void __launch_bounds__(kThreads, 1)
awe_gemm_wide_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ GemmParams p) {
    const uint32_t rank = ptx::cluster_ctarank();
    const int worker = (int)(blockIdx.x >> 1), num_workers = (int)(gridDim.x >> 1);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    uint8_t* after_tiles = smem_raw + (tiles_base - raw) + (size_t)kStages * kStageBytes;
    SharedW* sh = reinterpret_cast<SharedW*>(after_tiles + (size_t)kEpiWarps * kStageWarpBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&sh->acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->acc_empty[b]), kEpiWarps * 2);
        }
        sh->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(&sh->tmem_base), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();
    ptx::tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    if (warp >= 2 && warp < 6) {  // constant block scales, as in the 32-bit kernel
        const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
        ptx::tmem_st_fill16(tmem + (lane_base << 16) + kSfaCol, p.sf_word);
        ptx::tmem_st_fill16(tmem + (lane_base << 16) + kSfbCol, p.sf_word);
        ptx::tmem_wait_st();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();

    const int num_tiles = p.tiles_m * p.tiles_n;
    const int chunks = (p.num_kblocks + p.chunk_kblocks - 1) / p.chunk_kblocks;

    if (warp == 0) {
        if (lane == 0) {  // ------------------------------------------------------------ TMA producer
            uint32_t it = 0;
            bool ok = true;
            for (int t = worker, tile_iter = 0; t < num_tiles && ok; t += num_workers, ++tile_iter) {
                int tm, tn;
                tile_coords(t, p.tiles_m, p.tiles_n, &tm, &tn);
                const int row_a = (tm * 2 + (int)rank) * kTileM;
                const int row_b = tn * kN + (int)rank * kBRows;
                for (int kk = 0; kk < p.r && ok; ++kk) {
                    const int k = product_at(kk, tile_iter, p.r);
                    for (int kb = 0; kb < p.num_kblocks; ++kb, ++it) {
                        const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                        if (!(ok = wait(sh, ptx::smem_u32(&sh->empty[s]), ph ^ 1u, p.status, 11))) break;
                        const uint32_t bar = ptx::smem_u32(&sh->full[s]);
                        const uint32_t a_dst = tiles_base + s * kStageBytes;
                        const int x = (p.kblock0 + kb) * kBlockKBytes;
                        if (rank == 0) ptx::mbar_arrive_expect_tx(bar, 2 * kStageBytes);
                        const uint32_t bar0 = ptx::map_to_cta(bar, 0);
                        ptx::tma_load_3d_pair(a_dst, &map_a, bar0, x, row_a, p.ia[k]);
                        ptx::tma_load_3d_pair(a_dst + kABytes, &map_b, bar0, x, row_b, p.ib[k]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {  // ----------------------------------------------- MMA issuer
            uint32_t it = 0, drains = 0;
            bool ok = true;
            for (int t = worker; t < num_tiles && ok; t += num_workers) {
                for (int k = 0; k < p.r && ok; ++k) {
                    for (int c = 0; c < chunks && ok; ++c, ++drains) {
                        const uint32_t ab = drains & 1u;
                        if (!(ok = wait(sh, ptx::smem_u32(&sh->acc_empty[ab]), ((drains >> 1) & 1u) ^ 1u, p.status, 12)))
                            break;
                        ptx::tc_fence_after();
                        const int kb_end = min(p.num_kblocks, (c + 1) * p.chunk_kblocks);
                        for (int kb = c * p.chunk_kblocks; kb < kb_end; ++kb, ++it) {
                            const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                            if (!(ok = wait(sh, ptx::smem_u32(&sh->full[s]), ph, p.status, 13))) break;
                            ptx::tc_fence_after();
                            const uint32_t a_addr = tiles_base + s * kStageBytes;
                            const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
                            const uint64_t b_desc = ptx::smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                ptx::mma_mxf4_pair(tmem + (ab ? kAcc1 : kAcc0), a_desc + 2u * j, b_desc + 2u * j, kIdesc,
                                                   tmem + kSfaCol, tmem + kSfbCol,
                                                   (kb > c * p.chunk_kblocks || j > 0) ? 1u : 0u);
                            ptx::mma_commit_pair(ptx::smem_u32(&sh->empty[s]), 3);
                        }
                        if (ok) ptx::mma_commit_pair(ptx::smem_u32(&sh->acc_full[ab]), 3);
                    }
                }
            }
        }
    } else {  // ------------------------------------------------------------------------- epilogue
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)half * 64u;
        uint8_t* stage = after_tiles + (size_t)(warp - 2) * kStageWarpBytes;
        uint32_t acc_empty_bar[2];
        for (int b = 0; b < 2; ++b) acc_empty_bar[b] = ptx::map_to_cta(ptx::smem_u32(&sh->acc_empty[b]), 0);
        uint32_t drains = 0;
        bool ok = true;
        for (int t = worker, tile_iter = 0; t < num_tiles && ok; t += num_workers, ++tile_iter) {
            int tm, tn;
            tile_coords(t, p.tiles_m, p.tiles_n, &tm, &tn);
            long long sum[64];
#pragma unroll
            for (int i = 0; i < 64; ++i) sum[i] = 0;
            for (int kk = 0; kk < p.r && ok; ++kk) {
                const int ell = p.ell[product_at(kk, tile_iter, p.r)];
                for (int c = 0; c < chunks && ok; ++c, ++drains) {
                    const uint32_t ab = drains & 1u;
                    ok = wait(sh, ptx::smem_u32(&sh->acc_full[ab]), (drains >> 1) & 1u, p.status, 14);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    const uint32_t ta = taddr + (ab ? kAcc1 : kAcc0);
                    drain_block64<0>(ta, sum, p.acc_scale, ell);
                    drain_block64<1>(ta, sum, p.acc_scale, ell);
                    release(acc_empty_bar[ab], lane, true);
                }
            }
            if (!ok) break;
            const long long row0 = (long long)(tm * 2 + (int)rank) * kTileM + quarter * 32;
            const int col0 = tn * kN + half * 64;
            const int rows_valid = (int)max(0ll, min(32ll, (long long)p.M - row0));
            if (p.out_mode == OUT_I64) {
                uint8_t* gbase = reinterpret_cast<uint8_t*>(p.C) + (row0 * p.ldc + col0) * 8;
#pragma unroll
                for (int blk = 0; blk < 4; ++blk) {  // 16 columns = 128 bytes per row
                    auto chunk = [&](int c) {
                        const long long o0 = sum[blk * 16 + c * 2] >> p.log2D;
                        const long long o1 = sum[blk * 16 + c * 2 + 1] >> p.log2D;
                        return make_uint4((uint32_t)o0, (uint32_t)(o0 >> 32), (uint32_t)o1, (uint32_t)(o1 >> 32));
                    };
                    store_rows_128b<8>(stage, lane, chunk, gbase + blk * 128, p.ldc * 8, rows_valid,
                                       (p.N - col0 - blk * 16) * 8, p.vec_store, false);
                }
            } else {  // OUT_I32: the host has checked that the result fits
                uint8_t* gbase = reinterpret_cast<uint8_t*>(p.C) + (row0 * p.ldc + col0) * 4;
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {  // 32 columns = 128 bytes per row
                    auto chunk = [&](int c) {
                        uint32_t o[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) o[j] = (uint32_t)(sum[blk * 32 + c * 4 + j] >> p.log2D);
                        return make_uint4(o[0], o[1], o[2], o[3]);
                    };
                    store_rows_128b<4>(stage, lane, chunk, gbase + blk * 128, p.ldc * 4, rows_valid,
                                       (p.N - col0 - blk * 32) * 4, p.vec_store, false);
                }
            }
        }
    }

    if (sh->abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem, kTmemCols);
    }
}

}  // namespace

namespace gemm {

int wide_b_box_rows() { return kBRows; }

awe_status_t launch_gemm_wide(awe_ctx* h, const CUtensorMap& ma, const CUtensorMap& mb, GemmParams& p, cudaStream_t st) {
    bool& attr_set = h->smem_attr_set[2];
    if (!attr_set) {
        if (cudaFuncSetAttribute(awe_gemm_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) !=
            cudaSuccess)
            return AWE_ERR_CUDA;
        attr_set = true;
    }
    p.tiles_m = (p.M + kTileM * 2 - 1) / (kTileM * 2);
    p.tiles_n = (p.N + kN - 1) / kN;
    p.status = h->status_dev;
    p.clock_probe = nullptr;
    const int workers = std::min(p.tiles_m * p.tiles_n, h->sm_count / 2);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(workers * 2));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, awe_gemm_wide_kernel, ma, mb, p);
    if (err != cudaSuccess) {
        if (getenv("AWE_DEBUG")) fprintf(stderr, "awe: wide GEMM launch failed: %s\n", cudaGetErrorString(err));
        return AWE_ERR_CUDA;
    }
    h->launches += 1;
    return AWE_OK;
}

}  // namespace gemm
}  // namespace awe

// FP4 products and fused integer reconstruction (Algorithm 1, third loop and last step).
//
// One persistent CTA per SM.  In the default variant two CTAs on neighbouring SMs form a pair
// (a cluster of two) that shares one 256 x 256 output tile: each CTA loads its own 128 rows of
// the A plane and its own 128 of the 256 rows of the B plane, CTA 0 issues one MMA for both
// (cta_group::2: the halves of B are exchanged by the hardware, which halves the shared-memory
// traffic per flop), and each CTA keeps and drains the 128 x 256 accumulator of its own rows.
// The single-CTA variant works on 128 x 256 tiles alone.  For every tile and every product
// k a CTA streams the K-major E2M1 planes alpha_k (A side) and beta_k (B side) through a TMA ->
// shared-memory ring, multiplies them with tcgen05.mma kind::mxf4 (block scales held constant)
// into an FP32 accumulator in tensor memory, and after every K segment (Section 3.4: short
// enough that each partial sum is an integer below 2^24, hence exact) the epilogue warps drain
// the accumulator, convert it to integers and add l_k times it to a register-resident 32-bit
// running sum.  After the last product the sum is shifted by log2 D (Definition 4.1) or reduced
// mod m (Section 5.3) and written once.
//
// Records that mix operand formats (Appendix A: two E4M3 products and one E2M1 product) run in the
// kMixed instantiation: an E4M3 product streams one-byte elements through the same ring and the
// same descriptors with tcgen05.mma kind::f8f6f4, and its accumulator holds the product itself.
//
// The kDerive instantiation stores only the limb planes of a record whose other planes are sums of two
// limbs (a_i + a_j): for such a product the producer brings the two limb tiles of each side into two
// consecutive stages, six extra warps add them nibble by nibble (E2M1 codes through a 256-entry table)
// into the first stage, and the MMAs run on the result; the paper's remark on the cost of producing
// planes (Section 6.1), measured.
//
// 32-bit wrap-around is deliberate: sum_k l_k P_k is computed modulo 2^32, which equals the
// true D*C whenever |D*C| < 2^31 (checked on the host), although single terms may exceed it.
//
// Warp roles: warp 0 lane 0 issues TMA loads, warp 1 lane 0 issues MMAs (warp 1 also owns the
// tensor-memory allocation), warps 2..9 are the epilogue (warp w reads TMEM lanes 32*(w%4)..+31
// and columns 128*((w-2)/4)..+127).
// Every wait is bounded: when one expires the CTA records the site in the status word, raises a
// shared abort flag and winds down normally.
#include <cuda.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <type_traits>

#include "gemm_common.cuh"

namespace awe {
using namespace gemm;
namespace {

constexpr int kTileN = 256;
// Accumulator columns per tensor-memory load of the epilogue (16 or 32); also the number of columns
// the two accumulators share.  16 measured 1.3 % (6-product record) to 2.6 % (residue records) faster
// than 32: the shared columns are handed back after a smaller load and fewer registers are live.
#ifndef AWE_DRAIN_COLS
#define AWE_DRAIN_COLS 16
#endif
#define AWE_ACC1_COL (256 - AWE_DRAIN_COLS)
#ifndef AWE_PAIR_STAGES
#define AWE_PAIR_STAGES 6
#endif
// Per-variant sizes: a CTA of a pair stages only half of the B tile.
template <bool kPair>
struct Cfg {
    static constexpr int kBRows = kPair ? kTileN / 2 : kTileN;
    static constexpr int kBBytes = kBRows * kBlockKBytes;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = kPair ? AWE_PAIR_STAGES : 4;
    static constexpr int kCtas = kPair ? 2 : 1;
    static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 8 * 4096 + 1024;
    // mxf4 instruction descriptor: E2M1 x E2M1, both K-major, UE8M0 scales, dense K = 64
    static constexpr uint32_t kIdesc = (1u << 7) | (1u << 10) | ((uint32_t)(kTileN >> 3) << 17) | (1u << 23) |
                                       ((uint32_t)((kTileM * kCtas) >> 4) << 24);
    // f8f6f4 instruction descriptor: E4M3 x E4M3 (format code 0), FP32 accumulator, both K-major, K = 32
    static constexpr uint32_t kIdescF8 =
        (1u << 4) | ((uint32_t)(kTileN >> 3) << 17) | ((uint32_t)((kTileM * kCtas) >> 4) << 24);
};
constexpr int kMaxStages = 6;
// Threads per CTA (the variant that forms sum planes adds six warps) and first epilogue warp.
template <bool kDerive> struct Roles {
    static constexpr int kThreadsCta = kDerive ? kThreadsDerive : kThreads;
    static constexpr int kEpiWarp0 = 2;
};
// Two accumulators of 256 columns and the columns of scale bytes do not fit 512 columns side by
// side, so accumulator 1 starts inside the last columns of accumulator 0.  The epilogue reads
// those shared columns first and releases them separately (overlap_free), which lets the MMAs of
// the next segment start while the rest of the previous accumulator is still being drained.
// Constant scale bytes: with a 16-column overlap the second accumulator ends at column 496 and both
// operands read their (identical) scales from the last 16 columns.
constexpr uint32_t kSfaMain = AWE_DRAIN_COLS == 32 ? gemm::kSfaCol : 496u, kSfbMain = 496u;
constexpr uint32_t kAccCol0 = 0;
constexpr uint32_t kAccCol1 = AWE_ACC1_COL;

struct Shared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t overlap_free;
    uint64_t formed[kMaxStages];  // kDerive: the stage's tiles are complete (sums formed), both CTAs
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
    uint8_t add_lo[256], add_hi[256];  // kDerive: E2M1 code of x + y for codes (x, y), in the low / high nibble
};


__device__ __forceinline__ bool bounded_wait(Shared* sh, uint32_t bar, uint32_t parity, unsigned int* status,
                                             int site) {
    return bounded_wait_ns(&sh->abort_flag, bar, parity, status, site, kWaitLimitNs);
}

// Self-test of the bounded wait: one warp waits, with a budget of limit_ns, on a barrier that
// nothing ever signals, so the wait must give up, record its status and let the kernel return.
__global__ void bounded_wait_selftest_kernel(unsigned int* status, unsigned long long limit_ns, int site) {
    __shared__ uint64_t bar;
    __shared__ volatile uint32_t abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bar), 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    bounded_wait_ns(&abort_flag, ptx::smem_u32(&bar), 0, status, site, limit_ns);
}

// Residue arithmetic in FP32 (Section 5.3).  Every quantity is an integer of magnitude below 2^22
// held exactly in a float; x mod m is taken without leaving the FP32 pipe: q = round(x / m) by the
// add-and-subtract-1.5*2^23 trick, r = x - q m by one exact FMA, and one correction step in each
// direction puts r into the symmetric range [lo, hi] = [-floor(m/2), ceil(m/2) - 1].
__device__ __forceinline__ float mod_symmetric(float x, float m, float inv_m, float lo, float hi) {
    const float magic = 12582912.0f;
    const float q = __fadd_rn(__fadd_rn(__fmul_rn(x, inv_m), magic), -magic);
    float r = __fmaf_rn(-q, m, x);
    r = r > hi ? r - m : r;
    r = r < lo ? r + m : r;
    return r;
}

// E2M1 code <-> doubled integer (Section 3.1): sign, two exponent bits, one mantissa bit.
__device__ __forceinline__ int e2m1_value(int code) {
    const int e = (code >> 1) & 3, m = code & 1;
    const int v = e ? (2 + m) << (e - 1) : m;
    return (code & 8) ? -v : v;
}
__device__ __forceinline__ int e2m1_code(int v) {
    const int a = v < 0 ? -v : v;
    const int mag = a <= 4 ? a : (a == 6 ? 5 : (a == 8 ? 6 : (a == 12 ? 7 : 0)));
    return mag | ((v < 0 && mag) ? 8 : 0);
}
// Nibble-wise sum of two words of eight E2M1 codes (every sum lies in S by construction of the record).
__device__ __forceinline__ uint32_t add_e2m1x8(uint32_t x, uint32_t y, const uint8_t* lo, const uint8_t* hi) {
    const uint32_t il = (x & 0x0F0F0F0Fu) | ((y << 4) & 0xF0F0F0F0u);
    const uint32_t ih = ((x >> 4) & 0x0F0F0F0Fu) | (y & 0xF0F0F0F0u);
    uint32_t z = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b)
        z |= (uint32_t)(lo[(il >> (8 * b)) & 255u] | hi[(ih >> (8 * b)) & 255u]) << (8 * b);
    return z;
}

struct EpiMath {
    int out_mode, m;
    float acc_scale;
    float mf, inv_m, lo, hi;  // modulus and its symmetric range as floats
    int reduce_each;          // reduce the running residue sum after every segment (very long K only)
    // Every product of a segment stays below 2^22 in magnitude: adding 1.5 * 2^23 / acc_scale to the
    // accumulator word leaves the integer product in the low mantissa bits, so the conversion is one
    // FP32 add and the constant's own bits are taken off the sums once per tile.
    int use_magic;
    float magic;
    uint32_t magic_bits;
};

// Drain 32 accumulator columns (block BLK of this thread's 128) and fold them into the running sums.
// When `early_bar` is non-zero these are the columns the two accumulators share: they are handed
// back to the MMA issuer as soon as they sit in registers, before any arithmetic.

constexpr int kDrainCols = AWE_DRAIN_COLS;  // accumulator columns per tensor-memory load of the epilogue
// kEpi selects the arithmetic at compile time: kEpiResidue = residue record without per-segment
// reduction (measured 5 % faster than deciding at run time: fewer values live beside the 128 running
// sums of a thread), kEpiAny = decided at run time from `em` (every other case; the same specialisation
// of the exact records measured 12 % slower -- the compiler spilled more, not less -- and is not kept).
enum EpiKind { kEpiAny = 1, kEpiResidue = 2 };
template <int BLK, int kEpi>
__device__ __forceinline__ void drain_block(uint32_t taddr, uint32_t (&sum)[128], const EpiMath& em, int ell,
                                            uint32_t early_bar = 0, int lane = 0, bool remote = false) {
    uint32_t v[kDrainCols];
    if (kDrainCols == 32) ptx::tmem_ld_32x32(taddr + BLK * kDrainCols, reinterpret_cast<uint32_t(&)[32]>(v));
    else ptx::tmem_ld_32x16(taddr + BLK * kDrainCols, reinterpret_cast<uint32_t(&)[16]>(v));
    ptx::tmem_wait_ld();
    if (early_bar) release(early_bar, lane, remote);
    if constexpr (kEpi == kEpiResidue) {
        const float magic = 12582912.0f;
        const float q_scale = em.acc_scale * em.inv_m, m_scaled = em.mf / em.acc_scale;
        const float lam = (float)ell * em.acc_scale;
#pragma unroll
        for (int i = 0; i < kDrainCols; ++i) {
            const float a = __uint_as_float(v[i]);
            const float q = __fadd_rn(__fmaf_rn(a, q_scale, magic), -magic);
            const float res = __fmaf_rn(-q, m_scaled, a);
            sum[BLK * kDrainCols + i] = __float_as_uint(__fmaf_rn(lam, res, __uint_as_float(sum[BLK * kDrainCols + i])));
        }
        return;
    }
    if (em.out_mode == OUT_RAW_F32) {
#pragma unroll
        for (int i = 0; i < kDrainCols; ++i) sum[BLK * kDrainCols + i] = __float_as_uint(__uint_as_float(v[i]) * em.acc_scale);
    } else if (em.m) {
        // Running sum kept as a float (exact: |ell| <= m/2, |residue| <= m/2 + 1, few terms).  The
        // accumulator holds P / acc_scale; the scale (a power of two) is folded into the constants:
        // q = round(P / m), residue / acc_scale = acc - q (m / acc_scale), sum += (ell acc_scale) * that.
        // No range correction here: a residue one step outside [-m/2, m/2] is still congruent.
        const float magic = 12582912.0f;
        const float q_scale = em.acc_scale * em.inv_m, m_scaled = em.mf / em.acc_scale;
        const float lam = (float)ell * em.acc_scale;
#pragma unroll
        for (int i = 0; i < kDrainCols; ++i) {
            const float a = __uint_as_float(v[i]);
            const float q = __fadd_rn(__fmaf_rn(a, q_scale, magic), -magic);
            const float res = __fmaf_rn(-q, m_scaled, a);
            float sf = __fmaf_rn(lam, res, __uint_as_float(sum[BLK * kDrainCols + i]));
            if (em.reduce_each) sf = mod_symmetric(sf, em.mf, em.inv_m, em.lo, em.hi);
            sum[BLK * kDrainCols + i] = __float_as_uint(sf);
        }
    } else if (em.use_magic) {
#pragma unroll
        for (int i = 0; i < kDrainCols; ++i)
            sum[BLK * kDrainCols + i] += (uint32_t)ell * __float_as_uint(__fadd_rn(__uint_as_float(v[i]), em.magic));
    } else {
#pragma unroll
        for (int i = 0; i < kDrainCols; ++i)
            sum[BLK * kDrainCols + i] += (uint32_t)ell * (uint32_t)__float2int_rn(__uint_as_float(v[i]) * em.acc_scale);
    }
}

// Blocks FIRST .. LAST-1 of this thread's columns, in order.
template <int FIRST, int LAST, int kEpi>
__device__ __forceinline__ void drain_rest(uint32_t taddr, uint32_t (&sum)[128], const EpiMath& em, int ell) {
    if constexpr (FIRST < LAST) {
        drain_block<FIRST, kEpi>(taddr, sum, em, ell);
        drain_rest<FIRST + 1, LAST, kEpi>(taddr, sum, em, ell);
    }
}

// kMixed: some products of the record multiply E4M3 planes (their own pair of tensor maps, 128
// elements per 128-byte K block, kind::f8f6f4 without block scales, accumulator = the product
// itself); the others are E2M1 products as above.  Pair variant only.
// kGrouped: the reconstruction is a weighted sum of cells whose own sums fit 32 bits (GemmParams::group_*).
// kDerive: products with ia2[k] >= 0 multiply sum planes formed in shared memory (pair variant only).
// kOut: the output element type the tile write-out is compiled for (kOutAny: chosen at run time).
// With all three write-outs in one kernel the compiler spills ten times as much of the running sums.
enum OutSel { kOutAny = -1, kOut32 = 0, kOut64 = 1, kOut16 = 2 };
template <bool kPair, bool kMixed, bool kGrouped, bool kDerive = false, int kEpi = kEpiAny, int kOut = kOutAny>
__global__ void __launch_bounds__(Roles<kDerive>::kThreadsCta, 1)
awe_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                const __grid_constant__ CUtensorMap map_a8, const __grid_constant__ CUtensorMap map_b8,
                const __grid_constant__ GemmParams p) {
    static_assert(kPair || !kMixed, "mixed-format records run on CTA pairs");
    static_assert(!kDerive || (kPair && !kMixed && !kGrouped), "sum planes are formed in the plain pair variant only");
    static_assert(kEpi == kEpiAny || (!kMixed && !kGrouped), "the special epilogue kinds serve plain records");
    using C = Cfg<kPair>;
    constexpr int kStages = C::kStages;
    constexpr int kStageBytes = C::kStageBytes;
    constexpr uint32_t kIdesc = C::kIdesc;
    // rank of this CTA inside its pair; workers are pairs (or single CTAs)
    const uint32_t rank = kPair ? ptx::cluster_ctarank() : 0u;
    const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int num_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    Shared* sh = reinterpret_cast<Shared*>(smem_raw + (tiles_base - raw) + (size_t)kStages * kStageBytes +
                                           (size_t)kEpiWarps * kStageWarpBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&sh->acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->acc_empty[b]), kEpiWarps * C::kCtas);
        }
        ptx::mbar_init(ptx::smem_u32(&sh->overlap_free), (kEpiWarps / 2) * C::kCtas);
        if (kDerive)
            for (int s = 0; s < kStages; ++s) ptx::mbar_init(ptx::smem_u32(&sh->formed[s]), kFormerWarps * C::kCtas);
        sh->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
        if (kMixed) {
            ptx::prefetch_tensormap(&map_a8);
            ptx::prefetch_tensormap(&map_b8);
        }
    }
    if (warp == 1) {
        if (kPair) {
            ptx::tmem_alloc_pair(ptx::smem_u32(&sh->tmem_base), kTmemCols);
            ptx::tmem_relinquish_pair();
        } else {
            ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), kTmemCols);
            ptx::tmem_relinquish();
        }
    }
    if (kDerive && threadIdx.x >= 256) {
        const int idx = (int)threadIdx.x - 256;  // codes (x, y) = (idx & 15, idx >> 4)
        const int code = e2m1_code(e2m1_value(idx & 15) + e2m1_value(idx >> 4));
        sh->add_lo[idx] = (uint8_t)code;
        sh->add_hi[idx] = (uint8_t)(code << 4);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (kPair) ptx::cluster_sync_all();  // the other CTA's barriers are initialised before anyone signals them
    ptx::tc_fence_after();
    const uint32_t tmem = sh->tmem_base;

    // Constant block scales: every byte of 32 columns x 128 lanes holds the same UE8M0 value,
    // so whatever bytes the MMA picks as scale factors, it reads that value.
    constexpr int kEpiWarp0 = Roles<kDerive>::kEpiWarp0;
    if (warp >= kEpiWarp0 && warp < kEpiWarp0 + 4) {
        const uint32_t lane_base = (uint32_t)(warp & 3) * 32u;
        ptx::tmem_st_fill16(tmem + (lane_base << 16) + kSfaMain, p.sf_word);
        ptx::tmem_st_fill16(tmem + (lane_base << 16) + kSfbMain, p.sf_word);
        ptx::tmem_wait_st();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();

    // CTA 0 measures the SM clock it actually ran at (cycles over wall time of the launch)
    unsigned long long probe_c0 = 0, probe_t0 = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        probe_c0 = clock64();
        probe_t0 = ptx::globaltimer_ns();
    }

    const int num_tiles = p.tiles_m * p.tiles_n;
    const int chunks = (p.num_kblocks + p.chunk_kblocks - 1) / p.chunk_kblocks;
    const int chunks8 = kMixed ? (p.num_kblocks8 + p.chunk_kblocks8 - 1) / p.chunk_kblocks8 : 0;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------------------- TMA producer
            uint32_t it = 0;
            bool ok = true;
            for (int t = worker, tile_iter = 0; t < num_tiles && ok; t += num_workers, ++tile_iter) {
                int tm, tn;
                tile_coords(t, p.tiles_m, p.tiles_n, &tm, &tn);
                const int row_a = (tm * C::kCtas + (int)rank) * kTileM;
                const int row_b = tn * kTileN + (int)rank * C::kBRows;
                for (int kk = 0; kk < p.r && ok; ++kk) {
                    const int k = product_at(kk, tile_iter, p.r);
                    const bool f8 = kMixed && p.fp8[k];
                    const int nkb = f8 ? p.num_kblocks8 : p.num_kblocks, kb_first = f8 ? p.kblock0_8 : p.kblock0;
                    for (int kb = 0; kb < nkb; ++kb, ++it) {
                        const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                        if (!(ok = bounded_wait(sh, ptx::smem_u32(&sh->empty[s]), ph ^ 1u, p.status, 1))) break;
                        const uint32_t bar = ptx::smem_u32(&sh->full[s]);
                        const uint32_t a_dst = tiles_base + s * kStageBytes;
                        const int x = (kb_first + kb) * kBlockKBytes;
                        if (kDerive) {
                            // every CTA counts its own bytes on its own barrier (its forming warps wait there);
                            // a product of sum planes fills a second stage with the tiles to be added
                            ptx::mbar_arrive_expect_tx(bar, kStageBytes);
                            ptx::tma_load_3d(a_dst, &map_a, bar, x, row_a, p.ia[k]);
                            ptx::tma_load_3d(a_dst + kABytes, &map_b, bar, x, row_b, p.ib[k]);
                            if (p.ia2[k] >= 0) {
                                ++it;
                                const uint32_t s2 = it % kStages, ph2 = (it / kStages) & 1u;
                                if (!(ok = bounded_wait(sh, ptx::smem_u32(&sh->empty[s2]), ph2 ^ 1u, p.status, 6))) break;
                                const uint32_t bar2 = ptx::smem_u32(&sh->full[s2]);
                                const uint32_t dst2 = tiles_base + s2 * kStageBytes;
                                ptx::mbar_arrive_expect_tx(bar2, kStageBytes);
                                ptx::tma_load_3d(dst2, &map_a, bar2, x, row_a, p.ia2[k]);
                                ptx::tma_load_3d(dst2 + kABytes, &map_b, bar2, x, row_b, p.ib2[k]);
                            }
                        } else if (kPair) {
                            // both CTAs report their bytes to CTA 0's barrier, which expects the sum
                            if (rank == 0) ptx::mbar_arrive_expect_tx(bar, 2 * kStageBytes);
                            const uint32_t bar0 = ptx::map_to_cta(bar, 0);
                            // each load names its tensor map directly (a pointer chosen at run time between
                            // two kernel parameters made every copy far slower)
                            if (f8) {
                                ptx::tma_load_3d_pair(a_dst, &map_a8, bar0, x, row_a, p.ia[k]);
                                ptx::tma_load_3d_pair(a_dst + kABytes, &map_b8, bar0, x, row_b, p.ib[k]);
                            } else {
                                ptx::tma_load_3d_pair(a_dst, &map_a, bar0, x, row_a, p.ia[k]);
                                ptx::tma_load_3d_pair(a_dst + kABytes, &map_b, bar0, x, row_b, p.ib[k]);
                            }
                        } else {
                            ptx::mbar_arrive_expect_tx(bar, kStageBytes);
                            ptx::tma_load_3d(a_dst, &map_a, bar, x, row_a, p.ia[k]);
                            ptx::tma_load_3d(a_dst + kABytes, &map_b, bar, x, row_b, p.ib[k]);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---------------------------------------------------------------- MMA issuer
            uint32_t it = 0, drains = 0;
            bool ok = true;
            // One accumulation segment: K blocks [kb0, kb_end) into the accumulator at acc_col.  The
            // operand format is a compile-time constant of the loop: a per-instruction test of a
            // run-time flag here slowed every instruction of either format by half.
            bool sum_planes = false;  // kDerive: the current product multiplies sums of two stored planes
            auto issue_segment = [&](auto is_f8, int kb0, int kb_end, uint32_t acc_col, bool carry) {
                constexpr bool kF8 = decltype(is_f8)::value;
                for (int kb = kb0; kb < kb_end; ++kb, ++it) {
                    const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                    if (kDerive) {
                        // the forming warps of both CTAs have passed (and, for sum planes, rewritten) the stage
                        if (!(ok = bounded_wait(sh, ptx::smem_u32(&sh->formed[s]), ph, p.status, 7))) break;
                        ptx::fence_acq_rel_cluster();
                    } else if (!(ok = bounded_wait(sh, ptx::smem_u32(&sh->full[s]), ph, p.status, 3))) {
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t a_addr = tiles_base + s * kStageBytes;
                    const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr);
                    const uint64_t b_desc = ptx::smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // 32 bytes further along K inside the swizzle row (64 E2M1 or 32 E4M3 elements)
                        const uint32_t acc = (carry || kb > kb0 || j > 0) ? 1u : 0u;
                        if (kF8)
                            ptx::mma_f8_pair(tmem + acc_col, a_desc + 2u * j, b_desc + 2u * j, C::kIdescF8, acc);
                        else if (kPair)
                            ptx::mma_mxf4_pair(tmem + acc_col, a_desc + 2u * j, b_desc + 2u * j, kIdesc,
                                               tmem + kSfaMain, tmem + kSfbMain, acc);
                        else
                            ptx::mma_mxf4(tmem + acc_col, a_desc + 2u * j, b_desc + 2u * j, kIdesc, tmem + kSfaMain,
                                          tmem + kSfbMain, acc);
                    }
                    // frees the stage in both CTAs of a pair
                    if (kPair) ptx::mma_commit_pair(ptx::smem_u32(&sh->empty[s]), 3);
                    else ptx::mma_commit(ptx::smem_u32(&sh->empty[s]));
                    if (kDerive && sum_planes) {  // the stage that held the tiles added in goes back as well
                        ++it;
                        ptx::mma_commit_pair(ptx::smem_u32(&sh->empty[it % kStages]), 3);
                    }
                }
            };
            for (int t = worker, tile_iter = 0; t < num_tiles && ok; t += num_workers, ++tile_iter) {
                for (int kk = 0; kk < p.r && ok; ++kk) {
                    const int k = product_at(kk, tile_iter, p.r);
                    const bool f8 = kMixed && p.fp8[k];
                    if (kDerive) sum_planes = p.ia2[k] >= 0;
                    const int nkb = f8 ? p.num_kblocks8 : p.num_kblocks;
                    const int ckb = f8 ? p.chunk_kblocks8 : p.chunk_kblocks;
                    const int nchunks = f8 ? chunks8 : chunks;
                    // products of one set (equal coefficient; the host merges only when K is a single
                    // segment) accumulate into the same accumulator and are drained once
                    const bool set_first = kk == 0 || p.set_id[product_at(kk - 1, tile_iter, p.r)] != p.set_id[k];
                    const bool set_last = kk + 1 == p.r || p.set_id[product_at(kk + 1, tile_iter, p.r)] != p.set_id[k];
                    for (int c = 0; c < nchunks && ok; ++c) {
                        // accumulator (drains & 1): its previous contents (two segments ago) fully drained,
                        // and the columns it shares with the other accumulator already read
                        const uint32_t ab = drains & 1u;
                        const uint32_t acc_col = ab ? kAccCol1 : kAccCol0;
                        if (set_first) {
                            if (!(ok = bounded_wait(sh, ptx::smem_u32(&sh->acc_empty[ab]), ((drains >> 1) & 1u) ^ 1u,
                                                    p.status, 2)))
                                break;
                            if (drains > 0 && !(ok = bounded_wait(sh, ptx::smem_u32(&sh->overlap_free),
                                                                  (drains - 1u) & 1u, p.status, 5)))
                                break;
                            ptx::tc_fence_after();
                        }
                        const int kb_end = min(nkb, (c + 1) * ckb);
                        if (kMixed && f8) issue_segment(std::true_type{}, c * ckb, kb_end, acc_col, !set_first);
                        else issue_segment(std::false_type{}, c * ckb, kb_end, acc_col, !set_first);
                        if (set_last) {
                            if (ok) {
                                if (kPair) ptx::mma_commit_pair(ptx::smem_u32(&sh->acc_full[ab]), 3);
                                else ptx::mma_commit(ptx::smem_u32(&sh->acc_full[ab]));
                            }
                            ++drains;
                        }
                    }
                }
            }
        }
    } else if (kDerive && warp >= kEpiWarp0 + kEpiWarps) {
        // -------------------------------------------------------------------- forming warps (kDerive)
        // They follow the producer's sequence of stages.  A stage of a plain product is only passed on;
        // for a product of sum planes the tiles of the following stage are added, 16 bytes at a time,
        // into the stage the MMAs will read (both tiles of a side were written by TMA with the same
        // swizzle, so the sum is elementwise on equal offsets).
        const int ftid = (int)threadIdx.x - 32 * (kEpiWarp0 + kEpiWarps);
        uint32_t formed_bar[kMaxStages];
        for (int s = 0; s < kStages; ++s) formed_bar[s] = ptx::map_to_cta(ptx::smem_u32(&sh->formed[s]), 0);
        uint32_t it = 0;
        bool ok = true;
        for (int t = worker, tile_iter = 0; t < num_tiles && ok; t += num_workers, ++tile_iter) {
            for (int kk = 0; kk < p.r && ok; ++kk) {
                const int k = product_at(kk, tile_iter, p.r);
                const bool sum = p.ia2[k] >= 0;
                for (int kb = 0; kb < p.num_kblocks && ok; ++kb, ++it) {
                    const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                    ok = __all_sync(0xffffffffu, bounded_wait(sh, ptx::smem_u32(&sh->full[s]), ph, p.status, 8));
                    if (!ok) break;
                    if (sum) {
                        ++it;
                        const uint32_t s2 = it % kStages, ph2 = (it / kStages) & 1u;
                        ok = __all_sync(0xffffffffu, bounded_wait(sh, ptx::smem_u32(&sh->full[s2]), ph2, p.status, 9));
                        if (!ok) break;
                        uint4* dst = reinterpret_cast<uint4*>(smem_raw + (tiles_base - raw) + (size_t)s * kStageBytes);
                        const uint4* src =
                            reinterpret_cast<const uint4*>(smem_raw + (tiles_base - raw) + (size_t)s2 * kStageBytes);
                        for (int c = ftid; c < kStageBytes / 16; c += 32 * kFormerWarps) {
                            const uint4 x = dst[c], y = src[c];
                            dst[c] = make_uint4(add_e2m1x8(x.x, y.x, sh->add_lo, sh->add_hi),
                                                add_e2m1x8(x.y, y.y, sh->add_lo, sh->add_hi),
                                                add_e2m1x8(x.z, y.z, sh->add_lo, sh->add_hi),
                                                add_e2m1x8(x.w, y.w, sh->add_lo, sh->add_hi));
                        }
                        ptx::fence_proxy_async();  // the MMAs read these bytes through the async proxy
                        release(formed_bar[s2], lane, true);  // keeps the unused barrier's phase in step
                    }
                    release(formed_bar[s], lane, true);
                }
            }
        }
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
        // -------------------------------------------------------------------- epilogue
        const int quarter = warp & 3, half = (warp - kEpiWarp0) >> 2;
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)half * 128u;
        const int m = p.modulus;
        // symmetric representative of each coefficient keeps |l_k * residue| below m^2 / 4
        const int m_hi = (m + 1) / 2 - 1;
        uint32_t drains = 0;
        bool ok = true;
        // this warp's 4 KB staging block for the tile write-out
        uint8_t* stage = smem_raw + (tiles_base - raw) + (size_t)kStages * kStageBytes + (size_t)(warp - kEpiWarp0) * kStageWarpBytes;
        // barriers the MMA issuer (CTA 0) waits on
        uint32_t acc_empty_bar[2], overlap_bar = ptx::smem_u32(&sh->overlap_free);
        for (int b = 0; b < 2; ++b) acc_empty_bar[b] = ptx::smem_u32(&sh->acc_empty[b]);
        if (kPair) {
            overlap_bar = ptx::map_to_cta(overlap_bar, 0);
            for (int b = 0; b < 2; ++b) acc_empty_bar[b] = ptx::map_to_cta(acc_empty_bar[b], 0);
        }
        EpiMath em = {};
        em.out_mode = p.out_mode;
        em.m = m;
        em.acc_scale = p.acc_scale;
        if (m) {
            em.mf = (float)m;
            em.inv_m = 1.0f / (float)m;
            em.lo = (float)(-(m / 2));
            em.hi = (float)m_hi;
            // |sum| <= terms * (m/2)^2 must stay below 2^22
            em.reduce_each = (long long)p.r * chunks * (m / 2 + 2) * (m / 2 + 2) >= (1ll << 22);
        }
        em.use_magic = kEpi == kEpiAny && p.small_sums && !m && !kGrouped && p.out_mode != OUT_RAW_F32;
        if (kEpi == kEpiResidue) em.reduce_each = 0;
        em.magic = 12582912.0f / em.acc_scale;
        em.magic_bits = __float_as_uint(em.magic);
        for (int t = worker, tile_iter = 0; t < num_tiles && ok; t += num_workers, ++tile_iter) {
            uint32_t sum[128];
#pragma unroll
            for (int i = 0; i < 128; ++i) sum[i] = 0;
            uint32_t magic_corr = 0;  // sum over this tile's drains of l_k * (bit pattern of the conversion constant)
            // ---- tile write-out.  This thread owns one row and 128 consecutive columns; the warp passes
            // every 128-byte row piece through its shared-memory staging block so that each store
            // instruction writes 4 rows x 128 contiguous bytes instead of 32 rows x 16 bytes.
            // 64-bit output: scale * (sum >> log2D), stored or added to what is there.  (The tile's position
            // is worked out where it is needed, so that it does not occupy registers during the drains.)
            auto write_i64 = [&](long long scale, bool add) {
                int tm, tn;
                tile_coords(t, p.tiles_m, p.tiles_n, &tm, &tn);
                const long long row0 = (long long)(tm * C::kCtas + (int)rank) * kTileM + quarter * 32;
                const int col0 = tn * kTileN + half * 128;
                const int rows_valid = (int)max(0ll, min(32ll, (long long)p.M - row0));
                uint8_t* gbase = reinterpret_cast<uint8_t*>(p.C) + (row0 * p.ldc + col0) * 8;
#pragma unroll
                for (int blk = 0; blk < 8; ++blk) {  // 16 columns = 128 bytes per row
                    auto chunk = [&](int c) {
                        const long long o0 = (long long)((int)sum[blk * 16 + c * 2] >> p.log2D) * scale;
                        const long long o1 = (long long)((int)sum[blk * 16 + c * 2 + 1] >> p.log2D) * scale;
                        return make_uint4((uint32_t)o0, (uint32_t)(o0 >> 32), (uint32_t)o1, (uint32_t)(o1 >> 32));
                    };
                    store_rows_128b<8>(stage, lane, chunk, gbase + blk * 128, p.ldc * 8, rows_valid,
                                       (p.N - col0 - blk * 16) * 8, p.vec_store, add);
                }
            };
            int flushed = 0;
            for (int kk = 0; kk < p.r && ok; ++kk) {
                const int k = product_at(kk, tile_iter, p.r);
                int ell = p.ell[k];
                if (m && ell > m_hi) ell -= m;
                const bool f8 = kMixed && p.fp8[k];
                if (kMixed) {
                    em.acc_scale = f8 ? 1.0f : p.acc_scale;
                    em.magic = 12582912.0f / em.acc_scale;
                    em.magic_bits = __float_as_uint(em.magic);
                }

                // the accumulator of a merged set is complete after its last product
                const bool set_last = kk + 1 == p.r || p.set_id[product_at(kk + 1, tile_iter, p.r)] != p.set_id[k];
                const int nchunks = set_last ? (f8 ? chunks8 : chunks) : 0;
                for (int c = 0; c < nchunks && ok; ++c, ++drains) {
                    const uint32_t ab = drains & 1u;
                    ok = bounded_wait(sh, ptx::smem_u32(&sh->acc_full[ab]), (drains >> 1) & 1u, p.status, 4);
                    ok = __all_sync(0xffffffffu, ok);  // the TMEM loads below need the whole warp
                    if (!ok) break;
                    ptx::tc_fence_after();
                    // The 32 columns shared by the two accumulators are the last block of accumulator 0
                    // (held by the warps of column half 1) and the first block of accumulator 1 (half 0):
                    // they are read first and handed back at once.
                    constexpr int kBlocks = 128 / kDrainCols;
                    if (ab == 0) {
                        drain_block<kBlocks - 1, kEpi>(taddr + kAccCol0, sum, em, ell, half == 1 ? overlap_bar : 0u, lane, kPair);
                        drain_rest<0, kBlocks - 1, kEpi>(taddr + kAccCol0, sum, em, ell);
                    } else {
                        drain_block<0, kEpi>(taddr + kAccCol1, sum, em, ell, half == 0 ? overlap_bar : 0u, lane, kPair);
                        drain_rest<1, kBlocks, kEpi>(taddr + kAccCol1, sum, em, ell);
                    }
                    release(acc_empty_bar[ab], lane, kPair);
                    if (em.use_magic) magic_corr += (uint32_t)ell * em.magic_bits;
                }
                if (kGrouped) {
                    // A group of the grouped reconstruction is complete when the next product belongs to
                    // another one (or there is none): its 32-bit sum goes out with the group's weight,
                    // stored by the first group of the tile and added by the later ones, while the MMAs of
                    // the next products run.
                    const bool last = kk + 1 == p.r;
                    if (ok && (last || p.group_id[product_at(kk + 1, tile_iter, p.r)] != p.group_id[k])) {
                        write_i64(p.group_scale[k], flushed > 0 || p.accumulate != 0);
                        ++flushed;
#pragma unroll
                        for (int i = 0; i < 128; ++i) sum[i] = 0;
                    }
                }
            }
            if (!ok) break;
            if (kGrouped) continue;  // everything has been written group by group
            int tm, tn;
            tile_coords(t, p.tiles_m, p.tiles_n, &tm, &tn);
            const long long row0 = (long long)(tm * C::kCtas + (int)rank) * kTileM + quarter * 32;  // first row of the warp
            const int col0 = tn * kTileN + half * 128;
            const int rows_valid = (int)max(0ll, min(32ll, (long long)p.M - row0));
            if (em.use_magic) {
#pragma unroll
                for (int i = 0; i < 128; ++i) sum[i] -= magic_corr;
            }
            if (m) {
                // residue sums are floats: one last reduction, then to integers in the symmetric range
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    sum[i] = __float_as_uint(mod_symmetric(__uint_as_float(sum[i]), em.mf, em.inv_m, em.lo, em.hi) +
                                             12582912.0f) - 0x4B400000u;  // float -> int
            }
            if ((kOut == kOutAny || kOut == kOut32) &&
                (p.out_mode == OUT_I32 || p.out_mode == OUT_RES_I32 || p.out_mode == OUT_RAW_F32)) {
                uint8_t* gbase = reinterpret_cast<uint8_t*>(p.C) + (row0 * p.ldc + col0) * 4;
#pragma unroll
                for (int blk = 0; blk < 4; ++blk) {  // 32 columns = 128 bytes per row
                    const bool shift = p.out_mode == OUT_I32;
                    auto chunk = [&](int c) {
                        uint32_t o[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t x = sum[blk * 32 + c * 4 + j];
                            o[j] = shift ? (uint32_t)((int)x >> p.log2D) : x;
                        }
                        return make_uint4(o[0], o[1], o[2], o[3]);
                    };
                    store_rows_128b<4>(stage, lane, chunk, gbase + blk * 128, p.ldc * 4, rows_valid,
                                       (p.N - col0 - blk * 32) * 4, p.vec_store, false);
                }
            } else if ((kOut == kOutAny || kOut == kOut64) && p.out_mode == OUT_I64) {
                write_i64(1, p.accumulate != 0);
            } else if (kOut == kOutAny || kOut == kOut16) {  // OUT_RES_I16
                uint8_t* gbase = reinterpret_cast<uint8_t*>(p.C) + (row0 * p.ldc + col0) * 2;
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {  // 64 columns = 128 bytes per row
                    auto chunk = [&](int c) {
                        uint32_t w[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            w[j] = (sum[blk * 64 + c * 8 + 2 * j] & 0xFFFFu) | (sum[blk * 64 + c * 8 + 2 * j + 1] << 16);
                        return make_uint4(w[0], w[1], w[2], w[3]);
                    };
                    store_rows_128b<2>(stage, lane, chunk, gbase + blk * 128, p.ldc * 2, rows_valid,
                                       (p.N - col0 - blk * 64) * 2, p.vec_store, false);
                }
            }
        }
    }

    // ------------------------------------------------------------------------ wind down
    if (sh->abort_flag) {
        // give copies and MMAs that are still in flight time to land before memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0 && p.clock_probe) {
        p.clock_probe[0] = clock64() - probe_c0;
        p.clock_probe[1] = ptx::globaltimer_ns() - probe_t0;
    }
    if (kPair) ptx::cluster_sync_all();  // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        ptx::tc_fence_after();
        if (kPair) ptx::tmem_dealloc_pair(tmem, kTmemCols);
        else ptx::tmem_dealloc(tmem, kTmemCols);
    }
}

// The pair variant is the default; AWE_GEMM_SINGLE_CTA=1 in the environment selects the other.
bool use_pairs() {
    static const bool v = [] {
        const char* e = getenv("AWE_GEMM_SINGLE_CTA");
        return !(e && e[0] == '1');
    }();
    return v;
}

template <bool kPair, bool kMixed, bool kGrouped = false, bool kDerive = false, int kEpi = kEpiAny, int kOut = kOutAny>
awe_status_t launch_variant(awe_ctx* h, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ma8,
                            const CUtensorMap& mb8, GemmParams& p, cudaStream_t st) {
    using C = Cfg<kPair>;
    bool& attr_set = h->smem_attr_set[(kOut + 1) * 8 + (kEpi == kEpiResidue ? 6 : (kDerive ? 5 : (kGrouped ? 4 : (kMixed ? 3 : (kPair ? 0 : 1)))))];
    if (!attr_set) {
        if (cudaFuncSetAttribute(awe_gemm_kernel<kPair, kMixed, kGrouped, kDerive, kEpi, kOut>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)C::kSmemBytes) != cudaSuccess)
            return AWE_ERR_CUDA;
        attr_set = true;
    }
    p.tiles_m = (p.M + kTileM * C::kCtas - 1) / (kTileM * C::kCtas);
    p.tiles_n = (p.N + kTileN - 1) / kTileN;
    p.status = h->status_dev;
    p.clock_probe = reinterpret_cast<unsigned long long*>(h->status_dev + 2);
    const int workers = std::min(p.tiles_m * p.tiles_n, h->sm_count / C::kCtas);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(workers * C::kCtas));
    cfg.blockDim = dim3(Roles<kDerive>::kThreadsCta);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C::kCtas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, awe_gemm_kernel<kPair, kMixed, kGrouped, kDerive, kEpi, kOut>, ma, mb, ma8, mb8, p);
    if (err != cudaSuccess) {
        if (getenv("AWE_DEBUG")) fprintf(stderr, "awe: GEMM launch failed: %s\n", cudaGetErrorString(err));
        return AWE_ERR_CUDA;
    }
    h->launches += 1;
    return AWE_OK;
}

awe_status_t launch_gemm(awe_ctx* h, const CUtensorMap& ma, const CUtensorMap& mb, GemmParams& p, cudaStream_t st) {
    if (p.grouped) return launch_variant<true, false, true>(h, ma, mb, ma, mb, p, st);
    bool derive = false;
    for (int k = 0; k < p.r; ++k) derive = derive || p.ia2[k] >= 0;
    if (derive) return launch_variant<true, false, false, true>(h, ma, mb, ma, mb, p, st);
    if (!use_pairs()) return launch_variant<false, false>(h, ma, mb, ma, mb, p, st);
    // the plain pair kernel is compiled per output type, residue records also with their own arithmetic
    if (p.modulus && (p.out_mode == OUT_RES_I16 || p.out_mode == OUT_RES_I32)) {
        const long long chunks = (p.num_kblocks + p.chunk_kblocks - 1) / p.chunk_kblocks, half_m = p.modulus / 2 + 2;
        if ((long long)p.r * chunks * half_m * half_m < (1ll << 22)) {  // no reduction needed between segments
            return p.out_mode == OUT_RES_I16
                       ? launch_variant<true, false, false, false, kEpiResidue, kOut16>(h, ma, mb, ma, mb, p, st)
                       : launch_variant<true, false, false, false, kEpiResidue, kOut32>(h, ma, mb, ma, mb, p, st);
        }
    }
    switch (p.out_mode) {
        case OUT_I64: return launch_variant<true, false, false, false, kEpiAny, kOut64>(h, ma, mb, ma, mb, p, st);
        case OUT_RES_I16: return launch_variant<true, false, false, false, kEpiAny, kOut16>(h, ma, mb, ma, mb, p, st);
        default: return launch_variant<true, false, false, false, kEpiAny, kOut32>(h, ma, mb, ma, mb, p, st);
    }
}

// Records with E4M3 products: (ma, mb) cover the E2M1 planes, (ma8, mb8) the E4M3 planes.
awe_status_t launch_gemm_mixed(awe_ctx* h, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ma8,
                               const CUtensorMap& mb8, GemmParams& p, cudaStream_t st) {
    if (p.out_mode == OUT_I64) return launch_variant<true, true, false, false, kEpiAny, kOut64>(h, ma, mb, ma8, mb8, p, st);
    return launch_variant<true, true, false, false, kEpiAny, kOut32>(h, ma, mb, ma8, mb8, p, st);
}

int b_box_rows() { return use_pairs() ? Cfg<true>::kBRows : Cfg<false>::kBRows; }

// UE8M0 scale 2^0 on both operands: the accumulator then holds (product of doubled integers)/4.
constexpr uint32_t kScaleWord = 0x7F7F7F7Fu;
constexpr float kAccScale = 4.0f;

}  // namespace
}  // namespace awe

using namespace awe;

extern "C" awe_status_t awe_gemm_planes(awe_handle_t h, int enc, int modulus, const void* planesA_dev,
                                        const void* planesB_dev, int64_t M, int64_t N, int64_t K, void* C_dev,
                                        awe_out_dtype_t out_dt, int64_t ldc, int64_t k_chunk, void* stream) {
    return gemm_planes_window(h, enc, modulus, PlaneWindow{planesA_dev, M, 0}, PlaneWindow{planesB_dev, N, 0}, M, N, K,
                              C_dev, out_dt, ldc, k_chunk, stream);
}

awe_status_t awe::gemm_planes_window(awe_ctx* h, int enc, int modulus, PlaneWindow wa, PlaneWindow wb, int64_t M,
                                     int64_t N, int64_t K, void* C_dev, awe_out_dtype_t out_dt, int64_t ldc,
                                     int64_t k_chunk, void* stream) {
    const void* planesA_dev = wa.base;
    const void* planesB_dev = wb.base;
    if (!h || !planesA_dev || !planesB_dev || !C_dev || M <= 0 || N <= 0 || K <= 0) return AWE_ERR_INVALID_ARG;
    if (wa.row0 < 0 || wa.row0 + M > wa.plane_rows || wb.row0 < 0 || wb.row0 + N > wb.plane_rows)
        return AWE_ERR_INVALID_ARG;
    // 32-bit tile counters and TMA coordinates: at most 2^31 bytes along a plane row and 2^30 tiles
    if (M > (1 << 30) || N > (1 << 30) || K > (1ll << 31)) return AWE_ERR_INVALID_ARG;
    if (((M + 127) / 128) * ((N + 127) / 128) > (1ll << 30)) return AWE_ERR_INVALID_ARG;
    if (ldc < N || k_chunk < 0 || (k_chunk % 256) != 0) return AWE_ERR_INVALID_ARG;
    if ((int)out_dt < 0 || (int)out_dt > 3) return AWE_ERR_INVALID_ARG;
    awe_encoding_desc d;
    awe_status_t s = awe_encoding_info(enc, modulus, &d);
    if (s != AWE_OK) return s;
    const bool residue = d.modulus != 0;
    if (residue != (out_dt == AWE_C_RES_I16 || out_dt == AWE_C_RES_I32)) return AWE_ERR_UNSUPPORTED;
    const size_t elem = out_dt == AWE_C_I64 ? 8 : (out_dt == AWE_C_RES_I16 ? 2 : 4);
    if ((uintptr_t)planesA_dev % 256 || (uintptr_t)planesB_dev % 256 || (uintptr_t)C_dev % elem)
        return AWE_ERR_ALIGNMENT;
    const int vec_store = ((uintptr_t)C_dev % 16 == 0) && (((size_t)ldc * elem) % 16 == 0);
    // |C| <= max|a| max|b| K must fit the output type
    const int64_t amax = std::max(std::abs(d.a_lo), std::abs(d.a_hi));
    const int64_t bmax = std::max(std::abs(d.b_lo), std::abs(d.b_hi));
    if (out_dt == AWE_C_I32 && !i32_output_fits(d, K)) return AWE_ERR_RANGE;
    // A forced segment longer than K* (a quarter of it for the residue form, whose epilogue works below
    // 2^22) would let FP32 partial sums leave the exact range of Section 3.4.
    if (k_chunk > (residue ? std::max<int64_t>(256, d.k_star / 4) : std::max<int64_t>(256, d.k_star))) return AWE_ERR_RANGE;

    const int64_t pitch = plane_pitch_bytes(K);
    // 64-bit running sums are needed when not even one 256-element K block keeps D*C within 32 bits
    static const bool force_wide = [] { const char* e = getenv("AWE_FORCE_WIDE_SUMS"); return e && e[0] == '1'; }();
    bool wide = !residue && (force_wide || needs_wide_sums(d));
    // The 12-product record of Appendix A is a sum over limb-pair cells, 2AB = sum_{k,l} 71^(k+l) T_kl
    // with T_kl = -7 P + 126 P' + 9 Q.  Every T_kl is even and |T_kl| <= 2 * 120^2 * K (the two-limb
    // halves a_2k + 9 a_2k+1 stay within 12 + 9 * 12), so each cell fits the 32-bit sums of the fast
    // kernel: the cells of equal weight form a group, and the tile's 64-bit result is the sum of the three
    // group sums (halved) with their weights 1, 71 and 5041, each added to C when its group is done.
    struct Group { int first, count, scale; };
    static const Group kFp16Groups[3] = {{0, 3, 1}, {3, 6, 71}, {9, 3, 5041}};
    const bool grouped = wide && !force_wide && enc == AWE_ENC_FP16SIG_AWE12 && out_dt == AWE_C_I64 && use_pairs();
    if (grouped) wide = false;
    if (wide && !use_pairs()) return AWE_ERR_UNSUPPORTED;
    // E4M3 planes (mixed-format records) come first in the buffer, with rows twice as long
    int n8a = 0, n8b = 0;
    while (n8a < d.n_planes_a && d.plane_bits_a[n8a] == 8) ++n8a;
    while (n8b < d.n_planes_b && d.plane_bits_b[n8b] == 8) ++n8b;
    const bool mixed = n8a > 0 || n8b > 0;
    if (mixed && (wide || residue || !use_pairs() || n8a == d.n_planes_a || n8b == d.n_planes_b))
        return AWE_ERR_UNSUPPORTED;
    // row 0 of the window in the first E2M1 plane and in the first E4M3 plane of each side
    const uint8_t* a4 = (const uint8_t*)planesA_dev + ((size_t)n8a * wa.plane_rows * 2 + (size_t)wa.row0) * pitch;
    const uint8_t* b4 = (const uint8_t*)planesB_dev + ((size_t)n8b * wb.plane_rows * 2 + (size_t)wb.row0) * pitch;
    const uint8_t* a8 = (const uint8_t*)planesA_dev + (size_t)wa.row0 * 2 * pitch;
    const uint8_t* b8 = (const uint8_t*)planesB_dev + (size_t)wb.row0 * 2 * pitch;
    CUtensorMap ma, mb, ma8, mb8;
    if ((s = make_plane_map(h, a4, M, pitch, d.n_planes_a - n8a, kTileM, &ma, wa.plane_rows)) != AWE_OK) return s;
    if ((s = make_plane_map(h, b4, N, pitch, d.n_planes_b - n8b, wide ? wide_b_box_rows() : b_box_rows(), &mb,
                            wb.plane_rows)) != AWE_OK)
        return s;
    if (mixed) {
        if ((s = make_plane_map(h, a8, M, 2 * pitch, n8a, kTileM, &ma8, wa.plane_rows)) != AWE_OK) return s;
        if ((s = make_plane_map(h, b8, N, 2 * pitch, n8b, Cfg<true>::kBRows, &mb8, wb.plane_rows)) != AWE_OK) return s;
    }

    GemmParams p = {};
    p.M = (int)M;
    p.N = (int)N;
    p.r = d.r;
    for (int k = 0; k < d.r; ++k) {
        p.fp8[k] = d.fp8[k];
        p.ia[k] = d.fp8[k] ? d.ia[k] : d.ia[k] - n8a;  // index inside the map of its own format
        p.ib[k] = d.fp8[k] ? d.ib[k] : d.ib[k] - n8b;
        p.ell[k] = d.ell[k];
    }
    bool derive = false;
    for (int k = 0; k < AWE_MAX_PRODUCTS; ++k) {
        p.ia2[k] = k < d.r ? d.ia2[k] : -1;
        p.ib2[k] = k < d.r ? d.ib2[k] : -1;
        if ((p.ia2[k] >= 0) != (p.ib2[k] >= 0)) return AWE_ERR_UNSUPPORTED;  // sums are formed on both sides or on none
        derive = derive || p.ia2[k] >= 0;
    }
    if (derive && (wide || grouped || mixed || residue || !use_pairs())) return AWE_ERR_UNSUPPORTED;
    p.log2D = d.log2D;
    p.modulus = d.modulus;
    p.out_mode = (int)out_dt;
    p.C = C_dev;
    p.ldc = ldc;
    p.vec_store = vec_store;
    p.acc_scale = kAccScale;
    p.sf_word = kScaleWord;
    // exact accumulation segment (Section 3.4): a multiple of 256 not above K*
    int64_t kc = k_chunk ? k_chunk : std::max<int64_t>(256, d.k_star / 256 * 256);
    // the residue epilogue works on partial sums below 2^22 (see mod_symmetric)
    if (residue) kc = std::min<int64_t>(kc, std::max<int64_t>(256, d.k_star / 4 / 256 * 256));
    p.chunk_kblocks = (int)std::min<int64_t>(kc / 256, 1 << 20);
    const int64_t total_kblocks = pitch / kBlockKBytes;
    if (wide) {
        p.kblock0 = 0;
        p.num_kblocks = (int)total_kblocks;
        p.accumulate = 0;
        return launch_gemm_wide(h, ma, mb, p, (cudaStream_t)stream);
    }
    // 64-bit results: K is cut into launches whose own result fits 32 bits, added in int64
    int64_t seg_kblocks = total_kblocks;
    if (out_dt == AWE_C_I64 && !residue) {
        int64_t seg = ((int64_t)1 << 30) / (amax * bmax * ((int64_t)1 << d.log2D));
        seg_kblocks = std::max<int64_t>(1, std::min(total_kblocks, seg / 256));
    }
    if (residue) seg_kblocks = total_kblocks;
    if (grouped) {
        // 2 cells per group at most: |sum| <= 2 * 2 * 120^2 * K_seg must stay below 2^31
        seg_kblocks = std::min<int64_t>(total_kblocks, (((int64_t)1 << 31) - 1) / (4 * 120 * 120) / 256);
        int gi = 0;
        for (const Group& g : kFp16Groups) {
            for (int k = g.first; k < g.first + g.count; ++k) {
                if (d.ell[k] % g.scale) return AWE_ERR_UNSUPPORTED;
                p.ell[k] = d.ell[k] / g.scale;
                p.group_id[k] = gi;
                p.group_scale[k] = g.scale;
            }
            ++gi;
        }
        p.grouped = 1;
    }
    // Section 3.4: products with the same coefficient can be accumulated together (n_g of them) before
    // the accumulator is drained, as long as n_g c_A c_B K stays in the exact range.  Only worth doing
    // where coefficients repeat (base-13: 9 products in 5 sets; the 12-product record: 9 sets; the
    // four-product residue schemes: 3 sets) and K is a single segment.
    for (int k = 0; k < d.r; ++k) p.set_id[k] = k;
    if (!wide) {
        auto same = [&](int x, int y) {
            return p.ell[x] == p.ell[y] && p.fp8[x] == p.fp8[y] && p.group_id[x] == p.group_id[y];
        };
        int ord[AWE_MAX_PRODUCTS], set_of[AWE_MAX_PRODUCTS], n = 0, n_sets = 0, n_g = 1;
        bool used[AWE_MAX_PRODUCTS] = {false};
        for (int k = 0; k < d.r; ++k) {
            if (used[k]) continue;
            int run = 0;
            for (int j = k; j < d.r; ++j)
                if (!used[j] && same(k, j)) {
                    used[j] = true;
                    set_of[n] = n_sets;
                    ord[n++] = j;
                    ++run;
                }
            n_g = std::max(n_g, run);
            ++n_sets;
        }
        const int64_t k_launch = std::min(seg_kblocks, total_kblocks) * 256;
        const int64_t exact_range = residue ? ((int64_t)1 << 22) : ((int64_t)1 << 24);
        if (n_g > 1 && k_launch <= (int64_t)p.chunk_kblocks * 256 &&
            (int64_t)n_g * d.c_a * d.c_b * k_launch < exact_range) {
            GemmParams q = p;
            for (int k = 0; k < d.r; ++k) {
                q.ia[k] = p.ia[ord[k]];
                q.ib[k] = p.ib[ord[k]];
                q.ell[k] = p.ell[ord[k]];
                q.fp8[k] = p.fp8[ord[k]];
                q.ia2[k] = p.ia2[ord[k]];
                q.ib2[k] = p.ib2[ord[k]];
                q.group_id[k] = p.group_id[ord[k]];
                q.group_scale[k] = p.group_scale[ord[k]];
                q.set_id[k] = set_of[k];
            }
            p = q;
        }
    }
    for (int64_t kb0 = 0; kb0 < total_kblocks; kb0 += seg_kblocks) {
        p.kblock0 = (int)kb0;
        p.num_kblocks = (int)std::min(seg_kblocks, total_kblocks - kb0);
        p.accumulate = kb0 > 0;
        {
            // largest |accumulator| at a drain: products of one set (n_g of them) over one segment
            int n_g = 1;
            for (int k = 0; k < d.r; ++k) {
                int run = 0;
                for (int j = 0; j < d.r; ++j) run += p.set_id[j] == p.set_id[k];
                n_g = std::max(n_g, run);
            }
            const int64_t seg_len = 256 * (int64_t)std::min(p.num_kblocks, p.chunk_kblocks);
            p.small_sums = (int64_t)n_g * d.c_a * d.c_b * seg_len < ((int64_t)1 << 22);
        }
        if (mixed) {
            // an E4M3 K block holds 128 elements, an E2M1 block 256
            p.kblock0_8 = 2 * p.kblock0;
            p.num_kblocks8 = 2 * p.num_kblocks;
            p.chunk_kblocks8 = 2 * p.chunk_kblocks;
            s = launch_gemm_mixed(h, ma, mb, ma8, mb8, p, (cudaStream_t)stream);
        } else {
            s = launch_gemm(h, ma, mb, p, (cudaStream_t)stream);
        }
        if (s != AWE_OK) return s;
    }
    return AWE_OK;
}

extern "C" awe_status_t awe_selftest_bounded_wait(awe_handle_t h, int64_t limit_us, void* stream) {
    if (!h || limit_us <= 0 || limit_us > 1000000) return AWE_ERR_INVALID_ARG;
    bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(h->status_dev, (unsigned long long)limit_us * 1000ull,
                                                                     1000);
    if (cudaGetLastError() != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

extern "C" awe_status_t awe_fp4_product_raw(awe_handle_t h, const void* planeX_dev, const void* planeY_dev,
                                            int64_t M, int64_t N, int64_t K, float* P_dev, int64_t ldp,
                                            void* stream) {
    if (!h || !planeX_dev || !planeY_dev || !P_dev || M <= 0 || N <= 0 || K <= 0 || ldp < N)
        return AWE_ERR_INVALID_ARG;
    if (M > (1 << 30) || N > (1 << 30) || K > (1ll << 30)) return AWE_ERR_INVALID_ARG;
    if ((uintptr_t)planeX_dev % 256 || (uintptr_t)planeY_dev % 256 || (uintptr_t)P_dev % 4) return AWE_ERR_ALIGNMENT;
    const int64_t pitch = plane_pitch_bytes(K);
    CUtensorMap ma, mb;
    awe_status_t s;
    if ((s = make_plane_map(h, planeX_dev, M, pitch, 1, kTileM, &ma)) != AWE_OK) return s;
    if ((s = make_plane_map(h, planeY_dev, N, pitch, 1, b_box_rows(), &mb)) != AWE_OK) return s;
    GemmParams p = {};
    p.M = (int)M;
    p.N = (int)N;
    p.r = 1;
    p.ell[0] = 1;
    for (int k = 0; k < AWE_MAX_PRODUCTS; ++k) p.ia2[k] = p.ib2[k] = -1;
    p.out_mode = OUT_RAW_F32;
    p.C = P_dev;
    p.ldc = ldp;
    p.vec_store = ((uintptr_t)P_dev % 16 == 0) && ((ldp * 4) % 16 == 0);
    p.acc_scale = kAccScale;
    p.sf_word = kScaleWord;
    p.num_kblocks = (int)(pitch / kBlockKBytes);
    p.chunk_kblocks = p.num_kblocks;
    return launch_gemm(h, ma, mb, p, (cudaStream_t)stream);
}

extern "C" awe_status_t awe_fp8_product_raw(awe_handle_t h, const void* planeX_dev, const void* planeY_dev,
                                            int64_t M, int64_t N, int64_t K, float* P_dev, int64_t ldp,
                                            void* stream) {
    if (!h || !planeX_dev || !planeY_dev || !P_dev || M <= 0 || N <= 0 || K <= 0 || ldp < N)
        return AWE_ERR_INVALID_ARG;
    if (M > (1 << 30) || N > (1 << 30) || K > (1ll << 30)) return AWE_ERR_INVALID_ARG;
    if ((uintptr_t)planeX_dev % 256 || (uintptr_t)planeY_dev % 256 || (uintptr_t)P_dev % 4) return AWE_ERR_ALIGNMENT;
    if (!use_pairs()) return AWE_ERR_UNSUPPORTED;
    const int64_t pitch8 = 2 * plane_pitch_bytes(K);
    CUtensorMap ma, mb;
    awe_status_t s;
    if ((s = make_plane_map(h, planeX_dev, M, pitch8, 1, kTileM, &ma)) != AWE_OK) return s;
    if ((s = make_plane_map(h, planeY_dev, N, pitch8, 1, Cfg<true>::kBRows, &mb)) != AWE_OK) return s;
    GemmParams p = {};
    p.M = (int)M;
    p.N = (int)N;
    p.r = 1;
    p.ell[0] = 1;
    for (int k = 0; k < AWE_MAX_PRODUCTS; ++k) p.ia2[k] = p.ib2[k] = -1;
    p.fp8[0] = 1;
    p.out_mode = OUT_RAW_F32;
    p.C = P_dev;
    p.ldc = ldp;
    p.vec_store = ((uintptr_t)P_dev % 16 == 0) && ((ldp * 4) % 16 == 0);
    p.acc_scale = kAccScale;
    p.sf_word = kScaleWord;
    p.num_kblocks = p.chunk_kblocks = 1;  // no E2M1 product in this launch
    p.num_kblocks8 = (int)(pitch8 / kBlockKBytes);
    p.chunk_kblocks8 = p.num_kblocks8;
    return launch_gemm_mixed(h, ma, mb, ma, mb, p, (cudaStream_t)stream);
}

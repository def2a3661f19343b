// Pieces shared by the two GEMM kernels (32-bit and 64-bit running sums): constants, launch
// parameters, bounded waits, tile order, the coalescing tile write-out and the tensor-map helper.
#pragma once
#include <cuda.h>

#include "awe_internal.h"
#include "ptx.cuh"

namespace awe {
namespace gemm {

constexpr int kTileM = 128;  // rows of A (and of the accumulator) per CTA
constexpr int kBlockKBytes = 128;  // 256 E2M1 elements: one 128-byte swizzle row
constexpr int kABytes = kTileM * kBlockKBytes;  // 16 KB

constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
// The variant that forms sum planes in shared memory adds six warps for that work (warps 10..15).
constexpr int kThreadsDerive = 512;
constexpr int kFormerWarps = 6;
constexpr int kStageWarpBytes = 4096;  // 32 rows x 128 bytes per epilogue warp for the write-out
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSfaCol = 480;  // 16 columns of constant scale bytes each for A and B
constexpr uint32_t kSfbCol = 496;

enum OutMode { OUT_I32 = 0, OUT_I64 = 1, OUT_RES_I16 = 2, OUT_RES_I32 = 3, OUT_RAW_F32 = 4 };

struct GemmParams {
    int M, N;
    int tiles_m, tiles_n;
    int kblock0;        // first 256-element K block of this launch
    int num_kblocks;    // K blocks of this launch
    int chunk_kblocks;  // K blocks per exact accumulation segment
    int r;
    int ia[AWE_MAX_PRODUCTS], ib[AWE_MAX_PRODUCTS], ell[AWE_MAX_PRODUCTS];
    int log2D, modulus;
    int out_mode, accumulate;
    void* C;
    long long ldc;
    unsigned int* status;
    unsigned long long* clock_probe;  // [0] SM cycles, [1] nanoseconds spent by CTA 0 in this launch
    int vec_store;     // C rows are 16-byte aligned: vector stores allowed
    float acc_scale;   // accumulator value -> product of doubled integers
    uint32_t sf_word;  // four copies of the UE8M0 scale byte
    // Mixed-format records only: products whose planes are E4M3 bytes (128 elements per K block)
    // Grouped reconstruction (64-bit output only): products with equal group_id form a group whose
    // sum fits 32 bits; the result is sum_g group_scale_g * (group sum >> log2D), each group added to
    // C as soon as it is complete.
    // Section 3.4: products with equal coefficient (and format, and group) share one accumulator; they
    // carry the same set_id and sit next to each other.  All distinct when nothing is merged.
    int set_id[AWE_MAX_PRODUCTS];
    int grouped;
    int group_id[AWE_MAX_PRODUCTS], group_scale[AWE_MAX_PRODUCTS];
    int fp8[AWE_MAX_PRODUCTS];
    int kblock0_8, num_kblocks8, chunk_kblocks8;
    // Sum planes formed in the kernel: product k multiplies (plane ia[k] + plane ia2[k]) of A by
    // (plane ib[k] + plane ib2[k]) of B when ia2[k] >= 0 (then ib2[k] >= 0 too); -1 otherwise.
    int ia2[AWE_MAX_PRODUCTS], ib2[AWE_MAX_PRODUCTS];
    // every accumulator of this launch stays below 2^22 in magnitude when it is drained (Section 3.4's bound
    // with the segment length of this launch): lets the epilogue convert with one FP32 add
    int small_sums;
};

constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s

// Wait for a phase of an mbarrier, but never for longer than limit_ns: when the budget runs out the
// first CTA to notice records AWE_ERR_TIMEOUT and the site in the status word, every role of this
// CTA sees the abort flag at its next poll, and the kernel winds down normally.
__device__ __forceinline__ bool bounded_wait_ns(volatile uint32_t* abort_flag, uint32_t bar, uint32_t parity,
                                                unsigned int* status, int site, uint64_t limit_ns) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = ptx::globaltimer_ns();
    uint32_t polls = 0;
    for (;;) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if ((++polls & 63u) == 0 && ptx::globaltimer_ns() - t0 > limit_ns) {
            if (atomicCAS(status, 0u, (unsigned)AWE_ERR_TIMEOUT) == 0u) status[1] = (unsigned)site;
            *abort_flag = 1;
            return false;
        }
    }
}

__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int* tm, int* tn) {
    constexpr int kGroupM = 8;
    const int per_group = kGroupM * tiles_n;
    const int group = t / per_group, in_group = t % per_group;
    const int first_m = group * kGroupM;
    const int gsize = min(tiles_m - first_m, kGroupM);
    *tm = first_m + in_group % gsize;
    *tn = in_group / gsize;
}

// Order of the products inside a tile: ascending on a worker's even tiles, descending on its odd
// ones, so the planes used last by one tile are the first the next tile asks L2 for.  The sum of
// the products does not depend on the order.
__device__ __forceinline__ int product_at(int kk, int tile_iter, int r) { return (tile_iter & 1) ? r - 1 - kk : kk; }

// All lanes of the warp have finished reading their TMEM columns: one arrival for the warp on a
// barrier of this CTA or, in a pair, of CTA 0 (cluster address).
__device__ __forceinline__ void release(uint32_t bar, int lane, bool remote) {
    ptx::tc_fence_before();
    __syncwarp();
    if (lane == 0) {
        if (remote) ptx::mbar_arrive_cluster(bar);
        else ptx::mbar_arrive(bar);
    }
}

// Write 32 rows x 128 bytes held one row per lane (chunk(c), c = 0..7, yields its 16-byte pieces) to global memory through a
// 4 KB shared-memory block (16-byte chunks XOR-swizzled by row so neither pass has bank conflicts):
// afterwards lane l holds chunk l%8 of rows l/8, l/8+4, ... and one store instruction covers 4 rows
// x 128 contiguous bytes.  bytes_valid (<= 128, may be <= 0) is how much of the row piece lies
// inside the matrix; pieces that are cut or rows that are not 16-byte aligned fall back to
// element-wise stores.  With `add64` the 8-byte elements are added to what is already there.
template <int elem, class ChunkFn>
__device__ __forceinline__ void store_rows_128b(uint8_t* stage, int lane, ChunkFn chunk, uint8_t* gbase,
                                                long long row_pitch, int rows_valid, int bytes_valid, int vec_ok,
                                                bool add64) {
    if (bytes_valid <= 0 || rows_valid <= 0) return;  // warp-uniform
#pragma unroll
    for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(stage + lane * 128 + ((c ^ (lane & 7)) << 4)) = chunk(c);
    __syncwarp();
    const int c = lane & 7;
    if (add64 && elem == 8 && vec_ok && c * 16 + 16 <= bytes_valid) {
        // adding to what is there: reductions at L2 (no value comes back, so no load latency is exposed;
        // integer addition, and no other CTA touches these addresses, so the result is exact and
        // deterministic)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = i * 4 + (lane >> 3);
            const uint4 v = *reinterpret_cast<const uint4*>(stage + r * 128 + ((c ^ (r & 7)) << 4));
            if (r >= rows_valid) continue;
            unsigned long long* dst = reinterpret_cast<unsigned long long*>(gbase + r * row_pitch + c * 16);
            atomicAdd(dst, ((unsigned long long)v.y << 32) | v.x);
            atomicAdd(dst + 1, ((unsigned long long)v.w << 32) | v.z);
        }
        __syncwarp();
        return;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = i * 4 + (lane >> 3);
        const uint4 v = *reinterpret_cast<const uint4*>(stage + r * 128 + ((c ^ (r & 7)) << 4));
        if (r >= rows_valid) continue;
        uint8_t* dst = gbase + r * row_pitch + c * 16;
        if (vec_ok && c * 16 + 16 <= bytes_valid) {
            if (add64) {
                const longlong2 old = *reinterpret_cast<const longlong2*>(dst);
                const long long a = (long long)(((unsigned long long)v.y << 32) | v.x) + old.x;
                const long long b = (long long)(((unsigned long long)v.w << 32) | v.z) + old.y;
                *reinterpret_cast<longlong2*>(dst) = make_longlong2(a, b);
            } else {
                *reinterpret_cast<uint4*>(dst) = v;
            }
        } else {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 16 / elem; ++e) {
                if (c * 16 + (e + 1) * elem > bytes_valid) continue;
                if (elem == 4) {
                    reinterpret_cast<uint32_t*>(dst)[e] = w[e];
                } else if (elem == 2) {
                    reinterpret_cast<uint16_t*>(dst)[e] = (uint16_t)(w[e >> 1] >> (16 * (e & 1)));
                } else {
                    const long long x = (long long)(((unsigned long long)w[2 * e + 1] << 32) | w[2 * e]);
                    long long* d = reinterpret_cast<long long*>(dst) + e;
                    *d = add64 ? *d + x : x;
                }
            }
        }
    }
    __syncwarp();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// planes: n_planes planes of `rows` rows of pitch bytes, plane j starting plane_rows rows after plane
// j - 1 (plane_rows = 0: the planes are dense, rows apart).  Box: 128 bytes of K x box_rows rows of one plane.
inline awe_status_t make_plane_map(awe_ctx* h, const void* planes, int64_t rows, int64_t pitch, int n_planes,
                            int box_rows, CUtensorMap* out, int64_t plane_rows = 0) {
    if (!h->encode_tiled) return AWE_ERR_CUDA;
    if (plane_rows == 0) plane_rows = rows;
    cuuint64_t dims[3] = {(cuuint64_t)pitch, (cuuint64_t)rows, (cuuint64_t)n_planes};
    cuuint64_t strides[2] = {(cuuint64_t)pitch, (cuuint64_t)pitch * (cuuint64_t)plane_rows};
    cuuint32_t box[3] = {(cuuint32_t)kBlockKBytes, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((EncodeTiledFn)h->encode_tiled)(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(planes),
                                                  dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? AWE_OK : AWE_ERR_CUDA;
}


// 64-bit running sums variant (awe_gemm_wide.cu): 256 x 128 tiles per CTA pair.
awe_status_t launch_gemm_wide(awe_ctx* h, const CUtensorMap& ma, const CUtensorMap& mb, GemmParams& p, cudaStream_t st);
int wide_b_box_rows();

}  // namespace gemm
}  // namespace awe

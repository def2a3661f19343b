// Encode kernels (Algorithm 1, first two loops): per-value table lookup, plane formation and
// E2M1 packing in one pass over the operand.  HBM-bound: 1 byte read and n_planes/2 bytes
// written per element.
//
// The per-byte table holds, for raw input byte b, a 64-bit word whose byte j carries the E2M1
// code of stored plane j in its low nibble.  Two neighbouring elements are merged with one OR
// (the odd element shifted left by 4), which yields the packed output byte of every plane at
// once; byte permutes then gather 4 such words into one 32-bit output word per plane.
#include <algorithm>

#include "awe_internal.h"

namespace awe {
namespace {

constexpr int kEncThreads = 256;
constexpr int kLutReplicas = 16;  // one replica per lane of a half-warp: 64-bit lookups never conflict
constexpr size_t kLutSmemBytes = 256 * kLutReplicas * sizeof(uint64_t);

__device__ __forceinline__ void load_lut(uint64_t* lut_s, const uint64_t* __restrict__ lut_g) {
    for (int i = threadIdx.x; i < 256 * kLutReplicas; i += blockDim.x) lut_s[i] = lut_g[i / kLutReplicas];
    __syncthreads();
}

// Packed bytes of all planes for the element pair (b0 even k, b1 odd k).
__device__ __forceinline__ uint64_t pair_word(const uint64_t* lut_s, int rep, uint32_t b0, uint32_t b1) {
    return lut_s[b0 * kLutReplicas + rep] | (lut_s[b1 * kLutReplicas + rep] << 4);
}

// Transpose 4 pair words into one 32-bit word per plane (4 consecutive output bytes of each plane).
template <int NP>
__device__ __forceinline__ void gather4(const uint64_t (&w)[4], uint32_t (&out)[NP]) {
    const uint32_t l0 = (uint32_t)w[0], l1 = (uint32_t)w[1], l2 = (uint32_t)w[2], l3 = (uint32_t)w[3];
    const uint32_t t01 = __byte_perm(l0, l1, 0x5140), t23 = __byte_perm(l2, l3, 0x5140);
    out[0] = __byte_perm(t01, t23, 0x5410);
    if (NP > 1) out[1 % NP] = __byte_perm(t01, t23, 0x7632);
    if (NP > 2) {
        const uint32_t u01 = __byte_perm(l0, l1, 0x7362), u23 = __byte_perm(l2, l3, 0x7362);
        out[2 % NP] = __byte_perm(u01, u23, 0x5410);
        if (NP > 3) out[3 % NP] = __byte_perm(u01, u23, 0x7632);
    }
    if (NP > 4) {
        const uint32_t h0 = (uint32_t)(w[0] >> 32), h1 = (uint32_t)(w[1] >> 32), h2 = (uint32_t)(w[2] >> 32),
                       h3 = (uint32_t)(w[3] >> 32);
        const uint32_t s01 = __byte_perm(h0, h1, 0x5140), s23 = __byte_perm(h2, h3, 0x5140);
        out[4 % NP] = __byte_perm(s01, s23, 0x5410);
        if (NP > 5) out[5 % NP] = __byte_perm(s01, s23, 0x7632);
        if (NP > 6) {
            const uint32_t v01 = __byte_perm(h0, h1, 0x7362), v23 = __byte_perm(h2, h3, 0x7362);
            out[6 % NP] = __byte_perm(v01, v23, 0x5410);
            if (NP > 7) out[7 % NP] = __byte_perm(v01, v23, 0x7632);
        }
    }
}

// 8 input bytes (two 32-bit words, ascending k) -> one output word per plane.
template <int NP>
__device__ __forceinline__ void encode8(const uint64_t* lut_s, int rep, uint32_t lo, uint32_t hi,
                                        uint32_t (&out)[NP]) {
    uint64_t w[4];
    w[0] = pair_word(lut_s, rep, lo & 0xFF, (lo >> 8) & 0xFF);
    w[1] = pair_word(lut_s, rep, (lo >> 16) & 0xFF, lo >> 24);
    w[2] = pair_word(lut_s, rep, hi & 0xFF, (hi >> 8) & 0xFF);
    w[3] = pair_word(lut_s, rep, (hi >> 16) & 0xFF, hi >> 24);
    gather4<NP>(w, out);
}

// Operand stored with the reduction index contiguous (A as M x K): a warp handles 1024
// consecutive k of one row, 32 per lane.
template <int NP>
__global__ void __launch_bounds__(kEncThreads)
encode_rxk_kernel(const int8_t* __restrict__ X, int64_t R, int64_t K, int64_t ld, const uint64_t* __restrict__ lut_g,
                  uint8_t* __restrict__ planes, int64_t pitch, int64_t plane_stride, int vec_ok) {
    extern __shared__ __align__(16) uint64_t lut_s[];
    load_lut(lut_s, lut_g);
    const int lane = threadIdx.x & 31, rep = lane & (kLutReplicas - 1);
    const int64_t Kp = pitch * 2;
    const int64_t chunks = (Kp + 1023) / 1024;
    const int64_t items = R * chunks;
    const int64_t warps_total = (int64_t)gridDim.x * (kEncThreads / 32);
    for (int64_t it = (int64_t)blockIdx.x * (kEncThreads / 32) + (threadIdx.x >> 5); it < items; it += warps_total) {
        const int64_t row = it / chunks, k0 = (it % chunks) * 1024 + lane * 32;
        if (k0 >= Kp) continue;
        uint32_t in[8];
        const int8_t* src = X + row * ld + k0;
        if (vec_ok && k0 + 32 <= K) {
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(src));
            const uint4 b = __ldg(reinterpret_cast<const uint4*>(src) + 1);
            in[0] = a.x; in[1] = a.y; in[2] = a.z; in[3] = a.w;
            in[4] = b.x; in[5] = b.y; in[6] = b.z; in[7] = b.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t word = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t k = k0 + i * 4 + j;
                    const uint32_t byte = (k < K) ? (uint32_t)(uint8_t)src[i * 4 + j] : 0u;
                    word |= byte << (8 * j);
                }
                in[i] = word;
            }
        }
        uint32_t o[4][NP];
#pragma unroll
        for (int g = 0; g < 4; ++g) encode8<NP>(lut_s, rep, in[2 * g], in[2 * g + 1], o[g]);
        uint8_t* dst = planes + row * pitch + k0 / 2;
#pragma unroll
        for (int j = 0; j < NP; ++j)
            *reinterpret_cast<uint4*>(dst + j * plane_stride) = make_uint4(o[0][j], o[1][j], o[2][j], o[3][j]);
    }
}

// Operand stored with the reduction index strided (B as K x N): a block transposes a tile of
// 128 k x 128 r through shared memory; each thread then encodes 64 consecutive k of one r.
constexpr int kTile = 128;

template <int NP>
__global__ void __launch_bounds__(kEncThreads)
encode_kxr_kernel(const int8_t* __restrict__ X, int64_t R, int64_t K, int64_t ld, const uint64_t* __restrict__ lut_g,
                  uint8_t* __restrict__ planes, int64_t pitch, int64_t plane_stride, int vec_ok) {
    extern __shared__ __align__(16) uint64_t smem_all[];
    uint64_t* lut_s = smem_all;
    uint8_t* tile = reinterpret_cast<uint8_t*>(smem_all) + kLutSmemBytes;  // [128 k][128 r]
    load_lut(lut_s, lut_g);
    const int t = threadIdx.x, rep = t & (kLutReplicas - 1);
    const int64_t Kp = pitch * 2;
    const int64_t tiles_k = Kp / kTile, tiles_r = (R + kTile - 1) / kTile;
    for (int64_t tid = blockIdx.x; tid < tiles_k * tiles_r; tid += gridDim.x) {
        const int64_t k0 = (tid % tiles_k) * kTile, r0 = (tid / tiles_k) * kTile;
        if (vec_ok && r0 + kTile <= R) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = i * 32 + (t >> 3), c16 = t & 7;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (k0 + row < K) v = __ldg(reinterpret_cast<const uint4*>(X + (k0 + row) * ld + r0) + c16);
                *reinterpret_cast<uint4*>(tile + row * kTile + c16 * 16) = v;
            }
        } else {
            for (int i = 0; i < kTile * kTile / kEncThreads; ++i) {
                const int idx = i * kEncThreads + t, row = idx / kTile, col = idx % kTile;
                int8_t v = 0;
                if (k0 + row < K && r0 + col < R) v = X[(k0 + row) * ld + r0 + col];
                tile[row * kTile + col] = (uint8_t)v;
            }
        }
        __syncthreads();
        const int rl = t & (kTile - 1), kh = t >> 7;
        const int64_t r = r0 + rl;
        uint32_t o[8][NP];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            uint32_t lo = 0, hi = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                lo |= (uint32_t)tile[(kh * 64 + g * 8 + j) * kTile + rl] << (8 * j);
                hi |= (uint32_t)tile[(kh * 64 + g * 8 + 4 + j) * kTile + rl] << (8 * j);
            }
            encode8<NP>(lut_s, rep, lo, hi, o[g]);
        }
        if (r < R) {
            uint8_t* dst = planes + r * pitch + (k0 + kh * 64) / 2;
#pragma unroll
            for (int j = 0; j < NP; ++j) {
                uint4* d = reinterpret_cast<uint4*>(dst + j * plane_stride);
                d[0] = make_uint4(o[0][j], o[1][j], o[2][j], o[3][j]);
                d[1] = make_uint4(o[4][j], o[5][j], o[6][j], o[7][j]);
            }
        }
        __syncthreads();
    }
}

template <int NP>
cudaError_t launch(awe_layout_t layout, const int8_t* X, int64_t R, int64_t K, int64_t ld, const uint64_t* lut,
                   uint8_t* planes, int64_t pitch, int64_t plane_stride, int vec_ok, int sm_count,
                   cudaStream_t stream) {
    if (layout == AWE_ROWMAJOR_RxK) {
        const int64_t items = R * ((pitch * 2 + 1023) / 1024);
        const int64_t blocks = std::min<int64_t>((items + 7) / 8, (int64_t)sm_count * 4);
        encode_rxk_kernel<NP><<<(unsigned)blocks, kEncThreads, kLutSmemBytes, stream>>>(X, R, K, ld, lut, planes,
                                                                                        pitch, plane_stride, vec_ok);
    } else {
        const size_t smem = kLutSmemBytes + kTile * kTile;
        static bool attr_set[AWE_MAX_PLANES + 1] = {false};
        if (!attr_set[NP]) {
            cudaError_t e = cudaFuncSetAttribute(encode_kxr_kernel<NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem);
            if (e != cudaSuccess) return e;
            attr_set[NP] = true;
        }
        const int64_t tiles = (pitch * 2 / kTile) * ((R + kTile - 1) / kTile);
        const int64_t blocks = std::min<int64_t>(tiles, (int64_t)sm_count * 4);
        encode_kxr_kernel<NP><<<(unsigned)blocks, kEncThreads, smem, stream>>>(X, R, K, ld, lut, planes, pitch,
                                                                              plane_stride, vec_ok);
    }
    return cudaGetLastError();
}

}  // namespace
}  // namespace awe

using namespace awe;

extern "C" awe_status_t awe_encode(awe_handle_t h, int enc, int modulus, awe_side_t side, const void* X_dev,
                                   awe_in_dtype_t dt, awe_layout_t layout, int64_t R, int64_t K, int64_t ld,
                                   void* planes_dev, void* stream) {
    if (!h || !X_dev || !planes_dev || R <= 0 || K <= 0) return AWE_ERR_INVALID_ARG;
    if (side != AWE_SIDE_A && side != AWE_SIDE_B) return AWE_ERR_INVALID_ARG;
    if (dt != AWE_I8 && dt != AWE_I4_IN_I8) return AWE_ERR_INVALID_ARG;
    if (layout != AWE_ROWMAJOR_RxK && layout != AWE_ROWMAJOR_KxR) return AWE_ERR_INVALID_ARG;
    if (ld < (layout == AWE_ROWMAJOR_RxK ? K : R)) return AWE_ERR_INVALID_ARG;
    if ((uintptr_t)planes_dev % 256) return AWE_ERR_ALIGNMENT;
    const SideTable* t;
    if (!get_side_table(enc, modulus, side, dt, &t)) return AWE_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t* lut;
    awe_status_t s = device_lut(h, enc, modulus, side, dt, st, &lut);
    if (s != AWE_OK) return s;
    const int64_t pitch = plane_pitch_bytes(K), plane_stride = R * pitch;
    const int vec_ok = ((uintptr_t)X_dev % 16 == 0) && (ld % 16 == 0);
    const int8_t* X = (const int8_t*)X_dev;
    uint8_t* P = (uint8_t*)planes_dev;
    cudaError_t e;
    switch (t->n_planes) {
        case 1: e = launch<1>(layout, X, R, K, ld, lut, P, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 2: e = launch<2>(layout, X, R, K, ld, lut, P, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 3: e = launch<3>(layout, X, R, K, ld, lut, P, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 4: e = launch<4>(layout, X, R, K, ld, lut, P, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 6: e = launch<6>(layout, X, R, K, ld, lut, P, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        default: return AWE_ERR_UNSUPPORTED;
    }
    if (e != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

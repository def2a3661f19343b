// Encode kernels (Algorithm 1, first two loops): per-value table lookup, plane formation and
// E2M1 packing in one pass over the operand.  HBM-bound: 1 byte read and n_planes/2 bytes
// written per element.
//
// The per-byte table holds, for raw input byte b, a 64-bit word whose byte j carries the E2M1
// code of stored plane j in its low nibble.  Two neighbouring elements (even k, odd k) are merged
// with one shift-add per 32-bit half (the odd element moves to the high nibbles), which yields
// the packed output byte of every plane at once; byte permutes then gather 4 such words into one
// 32-bit output word per plane.  In shared memory every table entry is 128 bytes wide and holds
// one 32-bit copy per lane, so a warp's data-dependent lookups never collide on a bank and cost
// one shared-memory wavefront each.  With 5 or 6 planes the codes of planes 4 and 5 ride in the
// (otherwise empty) high nibbles of bytes 0 and 1 of that word; with 7 or 8 planes the entry is the
// full 64-bit word, 16 copies.
#include <algorithm>

#include "awe_internal.h"

namespace awe {
namespace {

constexpr int kEncThreads = 256;
constexpr size_t kLutSmemBytes = 256 * 128;
#ifndef AWE_KXR_LANES_K
#define AWE_KXR_LANES_K 4
#endif
constexpr int kKxrLanesK = AWE_KXR_LANES_K;            // lanes side by side along k
constexpr int kKxrRows = (32 / kKxrLanesK) * 4;       // r per warp item
constexpr int kKxrK = kKxrLanesK * 32;                // k per warp item

template <int NP>
__device__ __forceinline__ void load_lut(unsigned char* lut_s, const uint64_t* __restrict__ lut_g) {
    if (NP > 6) {
        uint64_t* d = reinterpret_cast<uint64_t*>(lut_s);
        for (int i = threadIdx.x; i < 256 * 16; i += blockDim.x) d[i] = lut_g[i >> 4];
    } else {
        uint32_t* d = reinterpret_cast<uint32_t*>(lut_s);
        // a warp reads 32 entries with one load and hands each to all lanes in turn
        const int lane = threadIdx.x & 31;
        for (int e0 = (threadIdx.x >> 5) * 32; e0 < 256; e0 += (blockDim.x >> 5) * 32) {
            const uint64_t e = lut_g[e0 + lane];
            // planes 0-3 stay in the low nibbles of bytes 0-3; planes 4, 5 move to the high nibbles of bytes 0, 1
            const uint32_t c = (uint32_t)e | (((uint32_t)(e >> 32) & 0x0F0Fu) << 4);
#pragma unroll
            for (int i = 0; i < 32; ++i) d[(e0 + i) * 32 + lane] = __shfl_sync(0xFFFFFFFFu, c, i);
        }
    }
    __syncthreads();
}

// Byte offset of this lane's private copy inside a 128-byte table entry.
template <int NP>
__device__ __forceinline__ uint32_t lane_slot(int lane) {
    return NP > 6 ? (uint32_t)(lane & 15) * 8u : (uint32_t)lane * 4u;
}

// Table words (low half: planes 0-3, high half: planes 4-7) of byte number I of `word`.
template <int NP, int I>
__device__ __forceinline__ uint2 lookup(const unsigned char* lut_s, uint32_t slot, uint32_t word) {
    // entry address = byte * 128; the lane slot occupies bits below 7 and is OR-ed in
    const uint32_t shifted = I == 0 ? (word << 7) : (word >> (8 * I - 7));
    const uint32_t off = (shifted & 0x7F80u) | slot;
    if (NP > 6) return *reinterpret_cast<const uint2*>(lut_s + off);
    return make_uint2(*reinterpret_cast<const uint32_t*>(lut_s + off), 0u);
}

// 8 input bytes (two 32-bit words, ascending k) -> one packed output word per plane.
template <int NP>
__device__ __forceinline__ void encode8(const unsigned char* lut_s, uint32_t slot, uint32_t w0, uint32_t w1,
                                        uint32_t (&out)[NP]) {
    const uint2 e0 = lookup<NP, 0>(lut_s, slot, w0), e1 = lookup<NP, 1>(lut_s, slot, w0);
    const uint2 e2 = lookup<NP, 2>(lut_s, slot, w0), e3 = lookup<NP, 3>(lut_s, slot, w0);
    const uint2 e4 = lookup<NP, 0>(lut_s, slot, w1), e5 = lookup<NP, 1>(lut_s, slot, w1);
    const uint2 e6 = lookup<NP, 2>(lut_s, slot, w1), e7 = lookup<NP, 3>(lut_s, slot, w1);
    // pair words: byte j = packed byte (even k low nibble, odd k high nibble) of plane j
    uint32_t l0, l1, l2, l3, h0 = 0, h1 = 0, h2 = 0, h3 = 0;
    if (NP <= 4) {
        l0 = (e1.x << 4) + e0.x; l1 = (e3.x << 4) + e2.x; l2 = (e5.x << 4) + e4.x; l3 = (e7.x << 4) + e6.x;
    } else if (NP <= 6) {
        // compact entries: low nibbles = planes 0-3, high nibbles of bytes 0, 1 = planes 4, 5
        const uint32_t m = 0x0F0F0F0Fu;
        l0 = (e0.x & m) | ((e1.x << 4) & ~m); l1 = (e2.x & m) | ((e3.x << 4) & ~m);
        l2 = (e4.x & m) | ((e5.x << 4) & ~m); l3 = (e6.x & m) | ((e7.x << 4) & ~m);
        h0 = ((e0.x >> 4) & 0x0F0Fu) | (e1.x & 0xF0F0u); h1 = ((e2.x >> 4) & 0x0F0Fu) | (e3.x & 0xF0F0u);
        h2 = ((e4.x >> 4) & 0x0F0Fu) | (e5.x & 0xF0F0u); h3 = ((e6.x >> 4) & 0x0F0Fu) | (e7.x & 0xF0F0u);
    } else {
        l0 = (e1.x << 4) + e0.x; l1 = (e3.x << 4) + e2.x; l2 = (e5.x << 4) + e4.x; l3 = (e7.x << 4) + e6.x;
        h0 = (e1.y << 4) + e0.y; h1 = (e3.y << 4) + e2.y; h2 = (e5.y << 4) + e4.y; h3 = (e7.y << 4) + e6.y;
    }
    const uint32_t t01 = __byte_perm(l0, l1, 0x5140), t23 = __byte_perm(l2, l3, 0x5140);
    out[0] = __byte_perm(t01, t23, 0x5410);
    if (NP > 1) out[1 % NP] = __byte_perm(t01, t23, 0x7632);
    if (NP > 2) {
        const uint32_t u01 = __byte_perm(l0, l1, 0x7362), u23 = __byte_perm(l2, l3, 0x7362);
        out[2 % NP] = __byte_perm(u01, u23, 0x5410);
        if (NP > 3) out[3 % NP] = __byte_perm(u01, u23, 0x7632);
    }
    if (NP > 4) {
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

// 32 consecutive elements of one plane row (8 words, ascending k) -> 16 packed bytes per plane.
template <int NP>
__device__ __forceinline__ void encode32_store(const unsigned char* lut_s, uint32_t slot, const uint32_t (&in)[8],
                                               uint8_t* dst, int64_t plane_stride) {
    uint32_t o[4][NP];
#pragma unroll
    for (int g = 0; g < 4; ++g) encode8<NP>(lut_s, slot, in[2 * g], in[2 * g + 1], o[g]);
#pragma unroll
    for (int j = 0; j < NP; ++j)
        *reinterpret_cast<uint4*>(dst + j * plane_stride) = make_uint4(o[0][j], o[1][j], o[2][j], o[3][j]);
}

// Mixed-format record (2 x FP8 + 1 x FP4, Appendix A): the table word of an input byte carries the
// E4M3 bytes of planes 0 and 1 in bytes 0 and 1 and the E2M1 code of plane 2 in the low nibble of
// byte 2.  32 consecutive elements of a row give 32 bytes of each E4M3 plane and 16 of the E2M1
// plane.  Row 0 of plane 0 is at `planes`, plane 1 follows 2 * plane_stride bytes later (plane_stride
// counts E2M1 rows of pitch bytes, an E4M3 row is twice as long), row 0 of plane 2 is at `planes4`.
__device__ __forceinline__ void encode32_store_mixed(const unsigned char* lut_s, uint32_t slot,
                                                     const uint32_t (&in)[8], uint8_t* planes, uint8_t* planes4,
                                                     int64_t plane_stride, int64_t row, int64_t k0, int64_t pitch) {
    uint32_t p0[8], p1[8], p2[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t w0 = in[2 * g], w1 = in[2 * g + 1];
        const uint32_t e0 = lookup<3, 0>(lut_s, slot, w0).x, e1 = lookup<3, 1>(lut_s, slot, w0).x;
        const uint32_t e2 = lookup<3, 2>(lut_s, slot, w0).x, e3 = lookup<3, 3>(lut_s, slot, w0).x;
        const uint32_t e4 = lookup<3, 0>(lut_s, slot, w1).x, e5 = lookup<3, 1>(lut_s, slot, w1).x;
        const uint32_t e6 = lookup<3, 2>(lut_s, slot, w1).x, e7 = lookup<3, 3>(lut_s, slot, w1).x;
        const uint32_t t01 = __byte_perm(e0, e1, 0x5140), t23 = __byte_perm(e2, e3, 0x5140);
        const uint32_t t45 = __byte_perm(e4, e5, 0x5140), t67 = __byte_perm(e6, e7, 0x5140);
        p0[2 * g] = __byte_perm(t01, t23, 0x5410);
        p1[2 * g] = __byte_perm(t01, t23, 0x7632);
        p0[2 * g + 1] = __byte_perm(t45, t67, 0x5410);
        p1[2 * g + 1] = __byte_perm(t45, t67, 0x7632);
        // E2M1 pairs: even k in the low nibble (byte 2 of the even word), odd k in the high nibble
        const uint32_t q01 = (e0 >> 16) | ((e1 >> 12) & 0xF0u), q23 = (e2 >> 16) | ((e3 >> 12) & 0xF0u);
        const uint32_t q45 = (e4 >> 16) | ((e5 >> 12) & 0xF0u), q67 = (e6 >> 16) | ((e7 >> 12) & 0xF0u);
        p2[g] = __byte_perm(__byte_perm(q01, q23, 0x0040), __byte_perm(q45, q67, 0x0040), 0x5410);
    }
    const int64_t pitch8 = 2 * pitch;
    uint8_t* d0 = planes + row * pitch8 + k0;
    uint8_t* d1 = d0 + 2 * plane_stride;
    uint8_t* d2 = planes4 + row * pitch + k0 / 2;
    *reinterpret_cast<uint4*>(d0) = make_uint4(p0[0], p0[1], p0[2], p0[3]);
    *reinterpret_cast<uint4*>(d0 + 16) = make_uint4(p0[4], p0[5], p0[6], p0[7]);
    *reinterpret_cast<uint4*>(d1) = make_uint4(p1[0], p1[1], p1[2], p1[3]);
    *reinterpret_cast<uint4*>(d1 + 16) = make_uint4(p1[4], p1[5], p1[6], p1[7]);
    *reinterpret_cast<uint4*>(d2) = make_uint4(p2[0], p2[1], p2[2], p2[3]);
}

// Operand stored with the reduction index contiguous (A as M x K): a warp handles 1024
// consecutive k of one row, 32 per lane.  kMixed: the mixed-format record above (NP = 3).
// kPacked: the operand holds two 4-bit values per byte (element e of the array in byte e/2, low
// nibble first); nibbles are spread to one per byte and then take the same route.
template <int NP, bool kMixed = false, bool kPacked = false>
__global__ void __launch_bounds__(kEncThreads)
encode_rxk_kernel(const int8_t* __restrict__ X, int64_t R, int64_t K, int64_t ld, const uint64_t* __restrict__ lut_g,
                  uint8_t* __restrict__ planes, uint8_t* __restrict__ planes4, int64_t pitch, int64_t plane_stride,
                  int vec_ok) {
    extern __shared__ __align__(128) unsigned char lut_s[];
    load_lut<NP>(lut_s, lut_g);
    const int lane = threadIdx.x & 31;
    const uint32_t slot = lane_slot<NP>(lane);
    const int64_t Kp = pitch * 2;
    const int64_t chunks = (Kp + 1023) / 1024;
    const int64_t items = R * chunks;
    const int64_t warps_total = (int64_t)gridDim.x * (kEncThreads / 32);
    for (int64_t it = (int64_t)blockIdx.x * (kEncThreads / 32) + (threadIdx.x >> 5); it < items; it += warps_total) {
        const int64_t row = it / chunks, k0 = (it % chunks) * 1024 + lane * 32;
        if (k0 >= Kp) continue;
        uint32_t in[8];
        const int8_t* src = kPacked ? X + (row * ld + k0) / 2 : X + row * ld + k0;
        if (kPacked && vec_ok && k0 + 32 <= K) {
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(src));
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t lo = w[i] & 0x0F0F0F0Fu, hi = (w[i] >> 4) & 0x0F0F0F0Fu;
                in[2 * i] = __byte_perm(lo, hi, 0x5140);
                in[2 * i + 1] = __byte_perm(lo, hi, 0x7362);
            }
        } else if (kPacked) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t word = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t k = k0 + i * 4 + j;
                    if (k < K) {
                        const int64_t e = row * ld + k;
                        word |= (((uint32_t)(uint8_t)X[e >> 1] >> (4 * (e & 1))) & 0xFu) << (8 * j);
                    }
                }
                in[i] = word;
            }
        } else if (vec_ok && k0 + 32 <= K) {
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
        if (kMixed) encode32_store_mixed(lut_s, slot, in, planes, planes4, plane_stride, row, k0, pitch);
        else encode32_store<NP>(lut_s, slot, in, planes + row * pitch + k0 / 2, plane_stride);
    }
}

// Operand stored with the reduction index strided (B as K x N).  A warp handles kKxrRows
// consecutive r by kKxrK consecutive k: kKxrLanesK neighbouring lanes own the same 4 rows and
// consecutive runs of 32 k.  Each lane loads the 32 words X[k][r..r+3] of its k run (a warp-wide
// load covers kKxrLanesK row segments of 128/kKxrLanesK bytes), transposes them in registers with
// byte permutes into 4 rows of 32 consecutive k, and encodes each row exactly like the kernel
// above.  The lanes of a group write adjacent 16-byte pieces in the same instruction, so whole
// 32-byte sectors are written at once (a sector left half written costs a fill from DRAM).
template <int NP, bool kMixed = false, bool kPacked = false>
__global__ void __launch_bounds__(kEncThreads)
encode_kxr_kernel(const int8_t* __restrict__ X, int64_t R, int64_t K, int64_t ld, const uint64_t* __restrict__ lut_g,
                  uint8_t* __restrict__ planes, uint8_t* __restrict__ planes4, int64_t pitch, int64_t plane_stride,
                  int vec_ok) {
    extern __shared__ __align__(128) unsigned char lut_s[];
    load_lut<NP>(lut_s, lut_g);
    const int lane = threadIdx.x & 31;
    const uint32_t slot = lane_slot<NP>(lane);
    const int64_t Kp = pitch * 2;
    const int64_t k_items = (Kp + kKxrK - 1) / kKxrK, r_items = (R + kKxrRows - 1) / kKxrRows;
    const int64_t items = k_items * r_items;
    const int64_t warps_total = (int64_t)gridDim.x * (kEncThreads / 32);
    for (int64_t it = (int64_t)blockIdx.x * (kEncThreads / 32) + (threadIdx.x >> 5); it < items; it += warps_total) {
        // neighbouring warps take neighbouring r blocks of the same k range: their loads share k rows
        const int64_t r0 = (it % r_items) * kKxrRows + (lane / kKxrLanesK) * 4;
        const int64_t k0 = (it / r_items) * kKxrK + (lane % kKxrLanesK) * 32;
        if (r0 >= R || k0 >= Kp) continue;
        uint32_t raw[32];  // raw[i] = bytes X[k0+i][r0..r0+3]
        if (kPacked && vec_ok && r0 + 4 <= R && k0 + 32 <= K) {
            // 4 elements = 2 bytes per k row
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const uint32_t w = __ldg(reinterpret_cast<const uint16_t*>(X + ((k0 + i) * ld + r0) / 2));
                raw[i] = __byte_perm(w & 0x0F0Fu, (w >> 4) & 0x0F0Fu, 0x5140);
            }
        } else if (kPacked) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                uint32_t word = 0;
                if (k0 + i < K) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (r0 + j < R) {
                            const int64_t e = (k0 + i) * ld + r0 + j;
                            word |= (((uint32_t)(uint8_t)X[e >> 1] >> (4 * (e & 1))) & 0xFu) << (8 * j);
                        }
                }
                raw[i] = word;
            }
        } else if (vec_ok && r0 + 4 <= R && k0 + 32 <= K) {
#pragma unroll
            for (int i = 0; i < 32; ++i) raw[i] = __ldg(reinterpret_cast<const uint32_t*>(X + (k0 + i) * ld + r0));
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                uint32_t word = 0;
                if (k0 + i < K) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (r0 + j < R) word |= (uint32_t)(uint8_t)X[(k0 + i) * ld + r0 + j] << (8 * j);
                }
                raw[i] = word;
            }
        }
        // 4x4 byte transposes: t[j][g] = the 4 bytes of row r0+j at k0+4g .. k0+4g+3
        uint32_t t[4][8];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            const uint32_t a = raw[4 * g], b = raw[4 * g + 1], c = raw[4 * g + 2], d = raw[4 * g + 3];
            const uint32_t ab_lo = __byte_perm(a, b, 0x5140), cd_lo = __byte_perm(c, d, 0x5140);
            const uint32_t ab_hi = __byte_perm(a, b, 0x7362), cd_hi = __byte_perm(c, d, 0x7362);
            t[0][g] = __byte_perm(ab_lo, cd_lo, 0x5410);
            t[1][g] = __byte_perm(ab_lo, cd_lo, 0x7632);
            t[2][g] = __byte_perm(ab_hi, cd_hi, 0x5410);
            t[3][g] = __byte_perm(ab_hi, cd_hi, 0x7632);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (r0 + j >= R) continue;
            if (kMixed) encode32_store_mixed(lut_s, slot, t[j], planes, planes4, plane_stride, r0 + j, k0, pitch);
            else encode32_store<NP>(lut_s, slot, t[j], planes + (r0 + j) * pitch + k0 / 2, plane_stride);
        }
    }
}

// ---- 16-bit elements (12 significant bits): the table has 4096 entries of 64 bits (32 KB of shared
// memory, one copy), indexed by the low 12 bits of the element.
constexpr size_t kLut16SmemBytes = 4096 * sizeof(uint64_t);

__device__ __forceinline__ uint2 lookup16(const unsigned char* lut_s, uint32_t byte_offset) {
    return *reinterpret_cast<const uint2*>(lut_s + byte_offset);
}

// 8 elements held as 4 words (two 16-bit elements per word, ascending k) -> one output word per plane.
template <int NP>
__device__ __forceinline__ void encode8_16(const unsigned char* lut_s, const uint32_t (&w)[4], uint32_t (&out)[NP]) {
    uint32_t lo[4], hi[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint2 e0 = lookup16(lut_s, (w[i] << 3) & 0x7FF8u);   // even k: bits 0-11 of the word
        const uint2 e1 = lookup16(lut_s, (w[i] >> 13) & 0x7FF8u);  // odd k: bits 16-27
        lo[i] = (e1.x << 4) + e0.x;
        hi[i] = (e1.y << 4) + e0.y;
    }
    const uint32_t t01 = __byte_perm(lo[0], lo[1], 0x5140), t23 = __byte_perm(lo[2], lo[3], 0x5140);
    out[0] = __byte_perm(t01, t23, 0x5410);
    if (NP > 1) out[1 % NP] = __byte_perm(t01, t23, 0x7632);
    if (NP > 2) {
        const uint32_t u01 = __byte_perm(lo[0], lo[1], 0x7362), u23 = __byte_perm(lo[2], lo[3], 0x7362);
        out[2 % NP] = __byte_perm(u01, u23, 0x5410);
        if (NP > 3) out[3 % NP] = __byte_perm(u01, u23, 0x7632);
    }
    if (NP > 4) {
        const uint32_t s01 = __byte_perm(hi[0], hi[1], 0x5140), s23 = __byte_perm(hi[2], hi[3], 0x5140);
        out[4 % NP] = __byte_perm(s01, s23, 0x5410);
        if (NP > 5) out[5 % NP] = __byte_perm(s01, s23, 0x7632);
        if (NP > 6) {
            const uint32_t v01 = __byte_perm(hi[0], hi[1], 0x7362), v23 = __byte_perm(hi[2], hi[3], 0x7362);
            out[6 % NP] = __byte_perm(v01, v23, 0x5410);
            if (NP > 7) out[7 % NP] = __byte_perm(v01, v23, 0x7632);
        }
    }
}

// 32 consecutive 16-bit elements of one plane row (16 words) -> 16 packed bytes per plane.
template <int NP>
__device__ __forceinline__ void encode32_16_store(const unsigned char* lut_s, const uint32_t (&in)[16], uint8_t* dst,
                                                  int64_t plane_stride) {
    uint32_t o[4][NP];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint32_t w[4] = {in[4 * g], in[4 * g + 1], in[4 * g + 2], in[4 * g + 3]};
        encode8_16<NP>(lut_s, w, o[g]);
    }
#pragma unroll
    for (int j = 0; j < NP; ++j)
        *reinterpret_cast<uint4*>(dst + j * plane_stride) = make_uint4(o[0][j], o[1][j], o[2][j], o[3][j]);
}

__device__ __forceinline__ void load_lut16(unsigned char* lut_s, const uint64_t* __restrict__ lut_g) {
    uint64_t* d = reinterpret_cast<uint64_t*>(lut_s);
    for (int i = threadIdx.x; i < 4096; i += blockDim.x) d[i] = lut_g[i];
    __syncthreads();
}

// 16-bit operand with the reduction index contiguous: a warp handles 1024 consecutive k of one row.
template <int NP>
__global__ void __launch_bounds__(kEncThreads)
encode16_rxk_kernel(const uint16_t* __restrict__ X, int64_t R, int64_t K, int64_t ld,
                    const uint64_t* __restrict__ lut_g, uint8_t* __restrict__ planes, int64_t pitch,
                    int64_t plane_stride, int vec_ok) {
    extern __shared__ __align__(128) unsigned char lut_s[];
    load_lut16(lut_s, lut_g);
    const int lane = threadIdx.x & 31;
    const int64_t Kp = pitch * 2;
    const int64_t chunks = (Kp + 1023) / 1024;
    const int64_t items = R * chunks;
    const int64_t warps_total = (int64_t)gridDim.x * (kEncThreads / 32);
    for (int64_t it = (int64_t)blockIdx.x * (kEncThreads / 32) + (threadIdx.x >> 5); it < items; it += warps_total) {
        const int64_t row = it / chunks, k0 = (it % chunks) * 1024 + lane * 32;
        if (k0 >= Kp) continue;
        uint32_t in[16];
        const uint16_t* src = X + row * ld + k0;
        if (vec_ok && k0 + 32 <= K) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 a = __ldg(reinterpret_cast<const uint4*>(src) + q);
                in[4 * q] = a.x; in[4 * q + 1] = a.y; in[4 * q + 2] = a.z; in[4 * q + 3] = a.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int64_t k = k0 + 2 * i;
                const uint32_t e0 = (k < K) ? (uint32_t)src[2 * i] : 0u;
                const uint32_t e1 = (k + 1 < K) ? (uint32_t)src[2 * i + 1] : 0u;
                in[i] = e0 | (e1 << 16);
            }
        }
        encode32_16_store<NP>(lut_s, in, planes + row * pitch + k0 / 2, plane_stride);
    }
}

// 16-bit operand with the reduction index strided (K x N): a lane owns 2 consecutive r and 32 k;
// 4 neighbouring lanes cover 128 consecutive k of the same rows, so stores fill whole sectors.
template <int NP>
__global__ void __launch_bounds__(kEncThreads)
encode16_kxr_kernel(const uint16_t* __restrict__ X, int64_t R, int64_t K, int64_t ld,
                    const uint64_t* __restrict__ lut_g, uint8_t* __restrict__ planes, int64_t pitch,
                    int64_t plane_stride, int vec_ok) {
    extern __shared__ __align__(128) unsigned char lut_s[];
    load_lut16(lut_s, lut_g);
    const int lane = threadIdx.x & 31;
    const int64_t Kp = pitch * 2;
    constexpr int kRows = (32 / kKxrLanesK) * 2;
    const int64_t k_items = (Kp + kKxrK - 1) / kKxrK, r_items = (R + kRows - 1) / kRows;
    const int64_t items = k_items * r_items;
    const int64_t warps_total = (int64_t)gridDim.x * (kEncThreads / 32);
    for (int64_t it = (int64_t)blockIdx.x * (kEncThreads / 32) + (threadIdx.x >> 5); it < items; it += warps_total) {
        const int64_t r0 = (it % r_items) * kRows + (lane / kKxrLanesK) * 2;
        const int64_t k0 = (it / r_items) * kKxrK + (lane % kKxrLanesK) * 32;
        if (r0 >= R || k0 >= Kp) continue;
        uint32_t raw[32];  // raw[i] = elements X[k0+i][r0], X[k0+i][r0+1]
        if (vec_ok && r0 + 2 <= R && k0 + 32 <= K) {
#pragma unroll
            for (int i = 0; i < 32; ++i) raw[i] = __ldg(reinterpret_cast<const uint32_t*>(X + (k0 + i) * ld + r0));
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                uint32_t word = 0;
                if (k0 + i < K) {
                    word = (uint32_t)X[(k0 + i) * ld + r0];
                    if (r0 + 1 < R) word |= (uint32_t)X[(k0 + i) * ld + r0 + 1] << 16;
                }
                raw[i] = word;
            }
        }
        uint32_t t0[16], t1[16];  // rows r0 and r0+1: 32 consecutive k each, two per word
#pragma unroll
        for (int g = 0; g < 16; ++g) {
            t0[g] = __byte_perm(raw[2 * g], raw[2 * g + 1], 0x5410);
            t1[g] = __byte_perm(raw[2 * g], raw[2 * g + 1], 0x7632);
        }
        encode32_16_store<NP>(lut_s, t0, planes + r0 * pitch + k0 / 2, plane_stride);
        if (r0 + 1 < R) encode32_16_store<NP>(lut_s, t1, planes + (r0 + 1) * pitch + k0 / 2, plane_stride);
    }
}

// Grid: kBlocksPerSm blocks per SM is what the tables allow (7 x 32 KB of shared memory).  Registers
// let fewer be resident at once (5 of the 6-plane RxK kernel, 3 of the transposing one) and the rest
// follow as a second wave; measured at 8192 x 8192 that is still faster for 5 planes and more and for
// every transposing kernel (60 against 76 us for 6 planes) than a grid of resident blocks only, while
// the RxK kernels of up to 4 planes gain 2-3 us from a grid of exactly the resident blocks.
constexpr int kBlocksPerSm = 7;

template <typename Kernel>
int resident_blocks(Kernel kernel, size_t smem) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kEncThreads, smem) != cudaSuccess || n < 1)
        n = kBlocksPerSm;
    return std::min(n, kBlocksPerSm);
}

template <int NP>
cudaError_t launch16(awe_layout_t layout, const uint16_t* X, int64_t R, int64_t K, int64_t ld, const uint64_t* lut,
                     uint8_t* planes, int64_t pitch, int64_t plane_stride, int vec_ok, int sm_count,
                     cudaStream_t stream) {
    const int64_t warps_per_block = kEncThreads / 32;
    constexpr int kRows = (32 / kKxrLanesK) * 2;
    const int64_t items = layout == AWE_ROWMAJOR_RxK
                              ? R * ((pitch * 2 + 1023) / 1024)
                              : ((pitch * 2 + kKxrK - 1) / kKxrK) * ((R + kRows - 1) / kRows);
    const int64_t blocks =
        std::min<int64_t>((items + warps_per_block - 1) / warps_per_block, (int64_t)sm_count * kBlocksPerSm);
    if (layout == AWE_ROWMAJOR_RxK)
        encode16_rxk_kernel<NP><<<(unsigned)blocks, kEncThreads, kLut16SmemBytes, stream>>>(X, R, K, ld, lut, planes, pitch,
                                                                                           plane_stride, vec_ok);
    else
        encode16_kxr_kernel<NP><<<(unsigned)blocks, kEncThreads, kLut16SmemBytes, stream>>>(X, R, K, ld, lut, planes, pitch,
                                                                                           plane_stride, vec_ok);
    return cudaGetLastError();
}

template <int NP, bool kMixed = false, bool kPacked = false>
cudaError_t launch(awe_layout_t layout, const int8_t* X, int64_t R, int64_t K, int64_t ld, const uint64_t* lut,
                   uint8_t* planes, uint8_t* planes4, int64_t pitch, int64_t plane_stride, int vec_ok, int sm_count,
                   cudaStream_t stream) {
    const int64_t warps_per_block = kEncThreads / 32;
    if (layout == AWE_ROWMAJOR_RxK) {
        static const int per_sm = (NP <= 4 && !kMixed)
                                      ? resident_blocks(encode_rxk_kernel<NP, kMixed, kPacked>, kLutSmemBytes)
                                      : kBlocksPerSm;
        const int64_t items = R * ((pitch * 2 + 1023) / 1024);
        const int64_t blocks = std::min<int64_t>((items + warps_per_block - 1) / warps_per_block, (int64_t)sm_count * per_sm);
        encode_rxk_kernel<NP, kMixed, kPacked><<<(unsigned)blocks, kEncThreads, kLutSmemBytes, stream>>>(
            X, R, K, ld, lut, planes, planes4, pitch, plane_stride, vec_ok);
    } else {
        const int64_t items = ((pitch * 2 + kKxrK - 1) / kKxrK) * ((R + kKxrRows - 1) / kKxrRows);
        const int64_t blocks =
            std::min<int64_t>((items + warps_per_block - 1) / warps_per_block, (int64_t)sm_count * kBlocksPerSm);
        encode_kxr_kernel<NP, kMixed, kPacked><<<(unsigned)blocks, kEncThreads, kLutSmemBytes, stream>>>(
            X, R, K, ld, lut, planes, planes4, pitch, plane_stride, vec_ok);
    }
    return cudaGetLastError();
}

}  // namespace
}  // namespace awe

using namespace awe;

extern "C" awe_status_t awe_encode(awe_handle_t h, int enc, int modulus, awe_side_t side, const void* X_dev,
                                   awe_in_dtype_t dt, awe_layout_t layout, int64_t R, int64_t K, int64_t ld,
                                   void* planes_dev, void* stream) {
    return encode_window(h, enc, modulus, side, X_dev, dt, layout, R, K, ld, PlaneWindow{planes_dev, R, 0}, stream);
}

awe_status_t awe::encode_window(awe_ctx* h, int enc, int modulus, awe_side_t side, const void* X_dev, awe_in_dtype_t dt,
                                awe_layout_t layout, int64_t R, int64_t K, int64_t ld, PlaneWindow win, void* stream) {
    void* planes_dev = const_cast<void*>(win.base);
    if (!h || !X_dev || !planes_dev || R <= 0 || K <= 0 || win.row0 < 0 || win.row0 + R > win.plane_rows)
        return AWE_ERR_INVALID_ARG;
    if (side != AWE_SIDE_A && side != AWE_SIDE_B) return AWE_ERR_INVALID_ARG;
    if ((int)dt < 0 || (int)dt > 6) return AWE_ERR_INVALID_ARG;
    if (layout != AWE_ROWMAJOR_RxK && layout != AWE_ROWMAJOR_KxR) return AWE_ERR_INVALID_ARG;
    if (dt == AWE_I4_PACKED && (ld & 1)) return AWE_ERR_INVALID_ARG;  // rows start on byte boundaries
    if (ld < (layout == AWE_ROWMAJOR_RxK ? K : R)) return AWE_ERR_INVALID_ARG;
    if ((uintptr_t)planes_dev % 256) return AWE_ERR_ALIGNMENT;
    const SideTable* t;
    if (!get_side_table(enc, modulus, side, dt, &t)) return AWE_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const uint64_t* lut;
    awe_status_t s = device_lut(h, enc, modulus, side, dt, st, &lut);
    if (s != AWE_OK) return s;
    const int64_t pitch = plane_pitch_bytes(K), plane_stride = win.plane_rows * pitch;
    // vector path: 16-byte loads along k (RxK) or 4-byte loads along r (KxR)
    const int64_t align = layout == AWE_ROWMAJOR_RxK ? 16 : 4;
    const int vec_ok = ((uintptr_t)X_dev % align == 0) && (ld % align == 0);
    // row 0 of this call inside plane 0; the E4M3 planes of the mixed record (which come first) have rows
    // twice as long, and its E2M1 plane starts after the two of them
    const bool mixed = t->bits[0] == 8;
    uint8_t* P = (uint8_t*)planes_dev + win.row0 * pitch * (mixed ? 2 : 1);
    uint8_t* P4 = mixed ? (uint8_t*)planes_dev + 4 * plane_stride + win.row0 * pitch : P;
    cudaError_t e;
    if (is_16bit(dt)) {
        if ((uintptr_t)X_dev % 2) return AWE_ERR_ALIGNMENT;
        const int vec16 = layout == AWE_ROWMAJOR_RxK ? (((uintptr_t)X_dev % 16 == 0) && (ld % 8 == 0))
                                                     : (((uintptr_t)X_dev % 4 == 0) && (ld % 2 == 0));
        if (t->n_planes == 6)
            e = launch16<6>(layout, (const uint16_t*)X_dev, R, K, ld, lut, P, pitch, plane_stride, vec16, h->sm_count, st);
        else if (t->n_planes == 4)
            e = launch16<4>(layout, (const uint16_t*)X_dev, R, K, ld, lut, P, pitch, plane_stride, vec16, h->sm_count, st);
        else
            return AWE_ERR_UNSUPPORTED;
        if (e != cudaSuccess) return AWE_ERR_CUDA;
        h->launches += 1;
        return AWE_OK;
    }
    const int8_t* X = (const int8_t*)X_dev;
    if (dt == AWE_I4_PACKED) {
        // vector path: 16-byte loads of 32 nibbles along k (RxK) or 2-byte loads of 4 nibbles along r (KxR)
        const int vp = layout == AWE_ROWMAJOR_RxK ? (((uintptr_t)X_dev % 16 == 0) && (ld % 32 == 0))
                                                  : (((uintptr_t)X_dev % 2 == 0) && (ld % 4 == 0));
        switch (t->n_planes) {
            case 2: e = launch<2, false, true>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vp, h->sm_count, st); break;
            case 3: e = launch<3, false, true>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vp, h->sm_count, st); break;
            case 4: e = launch<4, false, true>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vp, h->sm_count, st); break;
            default: return AWE_ERR_UNSUPPORTED;
        }
        if (e != cudaSuccess) return AWE_ERR_CUDA;
        h->launches += 1;
        return AWE_OK;
    }
    if (t->bits[0] == 8) {
        e = launch<3, true>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vec_ok, h->sm_count, st);
        if (e != cudaSuccess) return AWE_ERR_CUDA;
        h->launches += 1;
        return AWE_OK;
    }
    switch (t->n_planes) {
        case 1: e = launch<1>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 2: e = launch<2>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 3: e = launch<3>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 4: e = launch<4>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        case 6: e = launch<6>(layout, X, R, K, ld, lut, P, P4, pitch, plane_stride, vec_ok, h->sm_count, st); break;
        default: return AWE_ERR_UNSUPPORTED;
    }
    if (e != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

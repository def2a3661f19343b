// Stand-alone reconstruction (Algorithm 1, last step): C = (sum_k l_k P_k) / D, or the same sum
// reduced mod m (Section 5.3), from r FP32 product matrices already in HBM -- the unfused form of
// what the GEMM kernel's epilogue does in registers.  One HBM pass: 4 r bytes read and one result
// written per element.
#include "awe_internal.h"

using namespace awe;

namespace {

struct ReconParams {
    int r;
    int ell[AWE_MAX_PRODUCTS];
    int log2D, modulus, out_dt;
    int wrap32;  // int32 output of a record whose products come with |D C| < 2^31: sums modulo 2^32 are exact
};

__device__ __forceinline__ int symmetric_mod(int x, int m) {
    int r = x % m;
    if (r < 0) r += m;
    return r > (m + 1) / 2 - 1 ? r - m : r;
}
__device__ __forceinline__ long long symmetric_mod(long long x, int m) {
    long long r = x % m;
    if (r < 0) r += m;
    return r > (m + 1) / 2 - 1 ? r - m : r;
}

// Thread per 4 consecutive columns of one row.  Aligned rows take the vector path: every 16-byte
// load of the r product matrices is issued before the first is used (r independent requests in
// flight per thread), the sums of the exact encodings with 32-bit output wrap modulo 2^32 exactly
// like the fused epilogue, and the four results leave as one 16-byte store (two for 64-bit output,
// one 8-byte store for 16-bit residues).
// R is the number of products as a compile-time constant (so that no predicated-off slot of a
// longer unrolled loop is issued), or 0 for any count up to AWE_MAX_PRODUCTS.
template <int R>
__global__ void __launch_bounds__(256, R > 0 && R <= 8 ? 3 : 2)
reconstruct_kernel(const float* __restrict__ P, long long plane_stride, long long ldp, int M, int N,
                   const __grid_constant__ ReconParams p, void* __restrict__ C, long long ldc, int vec_ld, int vec_st) {
    const int groups_per_row = (N + 3) / 4;
    const long long total = (long long)M * groups_per_row;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < total;
         g += (long long)gridDim.x * blockDim.x) {
        const int row = (int)(g / groups_per_row), col = (int)(g % groups_per_row) * 4;
        const int n = min(4, N - col);
        const float* src0 = P + (long long)row * ldp + col;
        constexpr int kSlots = R > 0 ? R : AWE_MAX_PRODUCTS;
        const int r = R > 0 ? R : p.r;
        float4 v[kSlots];
        if (vec_ld && n == 4) {
#pragma unroll
            for (int k = 0; k < kSlots; ++k)
                if (k < r) v[k] = __ldcs(reinterpret_cast<const float4*>(src0 + k * plane_stride));
        } else {
#pragma unroll
            for (int k = 0; k < kSlots; ++k)
                if (k < r) {
                    const float* src = src0 + k * plane_stride;
                    v[k].x = src[0];
                    v[k].y = n > 1 ? src[1] : 0.f;
                    v[k].z = n > 2 ? src[2] : 0.f;
                    v[k].w = n > 3 ? src[3] : 0.f;
                }
        }
        long long out[4];
        if (p.wrap32) {
            // |D C| < 2^31, so sums taken modulo 2^32 equal D C although single terms may not fit
            uint32_t acc[4] = {0, 0, 0, 0};
#pragma unroll
            for (int k = 0; k < kSlots; ++k)
                if (k < r) {
                    const uint32_t l = (uint32_t)p.ell[k];
                    acc[0] += l * (uint32_t)__float2int_rn(v[k].x);
                    acc[1] += l * (uint32_t)__float2int_rn(v[k].y);
                    acc[2] += l * (uint32_t)__float2int_rn(v[k].z);
                    acc[3] += l * (uint32_t)__float2int_rn(v[k].w);
                }
#pragma unroll
            for (int j = 0; j < 4; ++j) out[j] = (long long)((int)acc[j] >> p.log2D);
        } else {
            long long acc[4] = {0, 0, 0, 0};
#pragma unroll
            for (int k = 0; k < kSlots; ++k)
                if (k < r) {
                    const float f[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        int pk = __float2int_rn(f[j]);  // an exact integer below 2^24
                        if (p.modulus) pk = (int)symmetric_mod(pk, p.modulus);
                        acc[j] += (long long)p.ell[k] * pk;
                    }
                }
#pragma unroll
            for (int j = 0; j < 4; ++j) out[j] = p.modulus ? symmetric_mod(acc[j], p.modulus) : (acc[j] >> p.log2D);
        }
        const long long idx = (long long)row * ldc + col;
        if (vec_st && n == 4) {
            if (p.out_dt == AWE_C_I64) {
                longlong2* dst = reinterpret_cast<longlong2*>(reinterpret_cast<long long*>(C) + idx);
                __stcs(dst, make_longlong2(out[0], out[1]));
                __stcs(dst + 1, make_longlong2(out[2], out[3]));
            } else if (p.out_dt == AWE_C_RES_I16) {
                const uint32_t lo = ((uint32_t)out[0] & 0xFFFFu) | ((uint32_t)out[1] << 16);
                const uint32_t hi = ((uint32_t)out[2] & 0xFFFFu) | ((uint32_t)out[3] << 16);
                __stcs(reinterpret_cast<uint2*>(reinterpret_cast<short*>(C) + idx), make_uint2(lo, hi));
            } else {
                __stcs(reinterpret_cast<int4*>(reinterpret_cast<int*>(C) + idx),
                       make_int4((int)out[0], (int)out[1], (int)out[2], (int)out[3]));
            }
        } else {
            for (int j = 0; j < n; ++j) {
                if (p.out_dt == AWE_C_I64) reinterpret_cast<long long*>(C)[idx + j] = out[j];
                else if (p.out_dt == AWE_C_RES_I16) reinterpret_cast<short*>(C)[idx + j] = (short)out[j];
                else reinterpret_cast<int*>(C)[idx + j] = (int)out[j];
            }
        }
    }
}

}  // namespace

extern "C" awe_status_t awe_reconstruct(awe_handle_t h, int enc, int modulus, const float* P_dev, int64_t plane_stride,
                                        int64_t ldp, int64_t M, int64_t N, void* C_dev, awe_out_dtype_t out_dt,
                                        int64_t ldc, void* stream) {
    if (!h || !P_dev || !C_dev || M <= 0 || N <= 0 || ldp < N || ldc < N || plane_stride < M * ldp)
        return AWE_ERR_INVALID_ARG;
    if (M > (1 << 30) || N > (1 << 30) || (int)out_dt < 0 || (int)out_dt > 3) return AWE_ERR_INVALID_ARG;
    awe_encoding_desc d;
    awe_status_t s = awe_encoding_info(enc, modulus, &d);
    if (s != AWE_OK) return s;
    if ((d.modulus != 0) != (out_dt == AWE_C_RES_I16 || out_dt == AWE_C_RES_I32)) return AWE_ERR_UNSUPPORTED;
    if ((uintptr_t)P_dev % 4) return AWE_ERR_ALIGNMENT;
    ReconParams p = {};
    p.r = d.r;
    for (int k = 0; k < d.r; ++k) p.ell[k] = d.ell[k];
    p.log2D = d.log2D;
    p.modulus = d.modulus;
    p.out_dt = (int)out_dt;
    p.wrap32 = d.modulus == 0 && out_dt == AWE_C_I32 && !needs_wide_sums(d);
    const int vec_ld = ((uintptr_t)P_dev % 16 == 0) && (ldp % 4 == 0) && (plane_stride % 4 == 0);
    const size_t elem = out_dt == AWE_C_I64 ? 8 : (out_dt == AWE_C_RES_I16 ? 2 : 4);
    const int vec_st = ((uintptr_t)C_dev % (4 * elem) == 0) && (ldc % 4 == 0);
    const long long total = M * ((N + 3) / 4);
    const unsigned blocks = (unsigned)std::min<long long>((total + 255) / 256, (long long)h->sm_count * 24);
    cudaStream_t st = (cudaStream_t)stream;
#define AWE_RECON(R_) \
    reconstruct_kernel<R_><<<blocks, 256, 0, st>>>(P_dev, plane_stride, ldp, (int)M, (int)N, p, C_dev, ldc, vec_ld, vec_st)
    switch (d.r) {
        case 1: AWE_RECON(1); break;
        case 3: AWE_RECON(3); break;
        case 4: AWE_RECON(4); break;
        case 6: AWE_RECON(6); break;
        case 8: AWE_RECON(8); break;
        case 9: AWE_RECON(9); break;
        case 12: AWE_RECON(12); break;
        default: AWE_RECON(0); break;
    }
#undef AWE_RECON
    if (cudaGetLastError() != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

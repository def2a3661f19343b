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
};

__device__ __forceinline__ long long symmetric_mod(long long x, int m) {
    long long r = x % m;
    if (r < 0) r += m;
    return r > (m + 1) / 2 - 1 ? r - m : r;
}

// Thread per 4 consecutive columns of one row: 16-byte loads from each P_k when aligned.
__global__ void __launch_bounds__(256)
reconstruct_kernel(const float* __restrict__ P, long long plane_stride, long long ldp, int M, int N,
                   const __grid_constant__ ReconParams p, void* __restrict__ C, long long ldc, int vec_ok) {
    const int groups_per_row = (N + 3) / 4;
    const long long total = (long long)M * groups_per_row;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < total;
         g += (long long)gridDim.x * blockDim.x) {
        const int row = (int)(g / groups_per_row), col = (int)(g % groups_per_row) * 4;
        const int n = min(4, N - col);
        long long acc[4] = {0, 0, 0, 0};
        for (int k = 0; k < p.r; ++k) {
            const float* src = P + k * plane_stride + (long long)row * ldp + col;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (vec_ok && n == 4) {
                const float4 f = __ldg(reinterpret_cast<const float4*>(src));
                v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
            } else {
                for (int j = 0; j < n; ++j) v[j] = src[j];
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                long long pk = (long long)__float2int_rn(v[j]);  // an exact integer below 2^24
                if (p.modulus) pk = symmetric_mod(pk, p.modulus);
                acc[j] += (long long)p.ell[k] * pk;
            }
        }
        for (int j = 0; j < n; ++j) {
            const long long x = p.modulus ? symmetric_mod(acc[j], p.modulus) : (acc[j] >> p.log2D);
            const long long idx = (long long)row * ldc + col + j;
            if (p.out_dt == AWE_C_I64) reinterpret_cast<long long*>(C)[idx] = x;
            else if (p.out_dt == AWE_C_RES_I16) reinterpret_cast<short*>(C)[idx] = (short)x;
            else reinterpret_cast<int*>(C)[idx] = (int)x;
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
    const int vec_ok = ((uintptr_t)P_dev % 16 == 0) && (ldp % 4 == 0) && (plane_stride % 4 == 0);
    const long long total = M * ((N + 3) / 4);
    const unsigned blocks = (unsigned)std::min<long long>((total + 255) / 256, (long long)h->sm_count * 16);
    reconstruct_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(P_dev, plane_stride, ldp, (int)M, (int)N, p, C_dev, ldc,
                                                                 vec_ok);
    if (cudaGetLastError() != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

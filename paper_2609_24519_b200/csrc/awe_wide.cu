// Exact product of wide-integer matrices through a residue number system (Section 5.3):
// residues of both operands modulo pairwise coprime moduli, one residue product per modulus on the
// FP4 kernels (mod-m schemes), reconstruction by the Chinese remainder theorem.  For input width 54
// (the FP64 significand) the built-in set has 22 moduli and needs 60 FP4 GEMMs.
#include <cmath>
#include <cstring>

#include "awe_internal.h"

using namespace awe;

namespace {

constexpr int kMaxModuli = 32;
// 5 one-product, 13 three-product and 4 four-product moduli; product = 2^122.86.
const int kWideModuli[] = {7, 8, 9, 11, 13, 41, 43, 47, 53, 59, 61, 67, 71, 73, 79, 83, 85, 89, 139, 149, 151, 157};
constexpr int kNumWideModuli = sizeof(kWideModuli) / sizeof(int);

typedef unsigned __int128 u128;
typedef __int128 i128;

struct ResidueParams {
    int n;
    // per modulus, as floats: m, 1/m, 2^14, 2^28, 2^42 mod m, and the symmetric range
    float mf[kMaxModuli], inv_m[kMaxModuli], c1f[kMaxModuli], c2f[kMaxModuli], c3f[kMaxModuli];
    float lo[kMaxModuli], hi[kMaxModuli];
};

// |x| < 2^56 as four 14-bit limbs l0..l3: |x| = l0 + l1 2^14 + l2 2^28 + l3 2^42.
struct Limbs14 {
    unsigned int l0, l1, l2, l3;
    bool neg;
};

__device__ __forceinline__ Limbs14 split14(long long x) {
    const unsigned long long ax = x < 0 ? (unsigned long long)(-x) : (unsigned long long)x;
    Limbs14 r;
    r.l0 = (unsigned int)ax & 0x3FFFu;
    r.l1 = (unsigned int)(ax >> 14) & 0x3FFFu;
    r.l2 = (unsigned int)(ax >> 28) & 0x3FFFu;
    r.l3 = (unsigned int)(ax >> 42) & 0x3FFFu;
    r.neg = x < 0;
    return r;
}

// x mod m in the symmetric range, on the FP32 pipe (twice the issue rate of 32-bit integer
// multiplies).  f holds the signed limbs as floats; s = f0 + f1 c1 + f2 c2 + f3 c3 is an integer below 2^24 in magnitude, hence
// exact; q = round(s / m) by adding and subtracting 1.5 * 2^23, r = s - q m by one exact FMA, and one
// correction each way puts r into [-floor(m/2), ceil(m/2) - 1] even if q was off by one.  Returns r
// as the low byte of (r + 1.5 * 2^23)'s bit pattern, i.e. r in two's complement.
__device__ __forceinline__ uint32_t symmetric_residue_f(const float (&f)[4], float m, float inv_m, float c1, float c2,
                                                        float c3, float lo, float hi) {
    const float magic = 12582912.0f;
    const float sres = __fmaf_rn(f[3], c3, __fmaf_rn(f[2], c2, __fmaf_rn(f[1], c1, f[0])));
    const float q = __fadd_rn(__fadd_rn(__fmul_rn(sres, inv_m), magic), -magic);
    float r = __fmaf_rn(-q, m, sres);
    r = r > hi ? r - m : r;
    r = r < lo ? r + m : r;
    return __float_as_uint(r + magic) & 0xFFu;
}

// X: `count` 64-bit integers; out[t * count + i] = symmetric residue of X[i] modulo m[t].
// A thread takes 4 consecutive elements so every store is a 4-byte word and a warp writes 128
// contiguous bytes per modulus.
__global__ void __launch_bounds__(256)
wide_residues_kernel(const long long* __restrict__ X, long long count, const __grid_constant__ ResidueParams p,
                     int8_t* __restrict__ out) {
    const long long groups = (count + 3) / 4;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < groups;
         g += (long long)gridDim.x * blockDim.x) {
        const long long i0 = g * 4;
        long long x[4] = {0, 0, 0, 0};
        if (i0 + 4 <= count) {
            const longlong2 a = __ldg(reinterpret_cast<const longlong2*>(X + i0));
            const longlong2 b = __ldg(reinterpret_cast<const longlong2*>(X + i0) + 1);
            x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
        } else {
            for (int j = 0; j < 4; ++j)
                if (i0 + j < count) x[j] = X[i0 + j];
        }
        float f[4][4];  // signed 14-bit limbs of the four elements
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const Limbs14 v = split14(x[j]);
            const float sgn = v.neg ? -1.0f : 1.0f;
            f[j][0] = sgn * (float)v.l0;
            f[j][1] = sgn * (float)v.l1;
            f[j][2] = sgn * (float)v.l2;
            f[j][3] = sgn * (float)v.l3;
        }
        const bool full = (i0 + 4 <= count) && ((count & 3) == 0);
#pragma unroll 2
        for (int t = 0; t < p.n; ++t) {
            const float m = p.mf[t], inv_m = p.inv_m[t], c1 = p.c1f[t], c2 = p.c2f[t], c3 = p.c3f[t];
            const float lo = p.lo[t], hi = p.hi[t];
            uint32_t word = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) word |= symmetric_residue_f(f[j], m, inv_m, c1, c2, c3, lo, hi) << (8 * j);
            int8_t* dst = out + (long long)t * count + i0;
            if (full) {
                *reinterpret_cast<uint32_t*>(dst) = word;
            } else {
                for (int j = 0; j < 4; ++j)
                    if (i0 + j < count) dst[j] = (int8_t)(word >> (8 * j));
            }
        }
    }
}

struct CrtParams {
    int n;
    int m[kMaxModuli];
    unsigned int w[kMaxModuli][4];  // W_t = (M/m_t) ((M/m_t)^-1 mod m_t) < 2^123 in four 32-bit limbs
    unsigned int M[4];              // M = prod m_t
    unsigned long long M_lo, M_hi, half_lo, half_hi;
    double M_as_double;
};

// res[t * count + i]: symmetric residues of the unknown integers modulo m_t.  The integer with
// -M/2 < x <= M/2 is x = sum_t r_t W_t mod M (textbook CRT) with r_t taken in [0, m_t).  The sum is
// formed limb by limb (four 64-bit accumulators of 32 x 32-bit products, no carries needed: 22 terms
// below 2^40 each), the quotient by M (< 2^13) is estimated in double precision, q M is subtracted
// limb by limb, carries are propagated once, and at most two corrections fix the estimate.
constexpr int kCrtBatch = 12;

// One element: x in (-M/2, M/2] from the four limb sums a0..a3 of sum_t r_t W_t.
__device__ __forceinline__ i128 crt_reduce(unsigned long long a0, unsigned long long a1, unsigned long long a2,
                                           unsigned long long a3, const CrtParams& p, i128 M, i128 half) {
    const double xd = ((double)a3 * 4294967296.0 + (double)a2) * 18446744073709551616.0 +
                      (double)a1 * 4294967296.0 + (double)a0;
    const long long q = (long long)floor(xd / p.M_as_double);
    // d_k = a_k - q M_k (|d_k| < 2^46), then x - q M = sum_k d_k 2^(32 k) with signed carries
    long long c = (long long)a0 - q * (long long)p.M[0];
    const unsigned long long r0 = (unsigned long long)c & 0xFFFFFFFFull;
    c = (c >> 32) + (long long)a1 - q * (long long)p.M[1];
    const unsigned long long r1 = (unsigned long long)c & 0xFFFFFFFFull;
    c = (c >> 32) + (long long)a2 - q * (long long)p.M[2];
    const unsigned long long r2 = (unsigned long long)c & 0xFFFFFFFFull;
    c = (c >> 32) + (long long)a3 - q * (long long)p.M[3];  // top limb: signed, |c| < 2^28, so its low 32 bits
    // placed at bit 96 give the right two's-complement value even when the estimate was one too large
    i128 x = (i128)(((u128)(unsigned long long)c << 96) | ((u128)r2 << 64) | ((u128)r1 << 32) | (u128)r0);
    if (x < 0) x += M;
    if (x >= M) x -= M;
    if (x > half) x -= M;
    return x;
}

// A thread takes two neighbouring elements: one 4-byte load per modulus (a warp reads whole 128-byte
// lines), all loads of a batch of kCrtBatch moduli in flight together (with one 2-byte load at a time
// the kernel was bound by load latency), and the two 128-bit results leave as one 32-byte sector.
__global__ void __launch_bounds__(256)
wide_crt_kernel(const short* __restrict__ res, long long count, const __grid_constant__ CrtParams p,
                long long* __restrict__ out) {
    const i128 M = (i128)(((u128)p.M_hi << 64) | p.M_lo);
    const i128 half = (i128)(((u128)p.half_hi << 64) | p.half_lo);
    const long long pairs = (count + 1) / 2;
    // every modulus' array starts on a 4-byte boundary
    const bool vec = (count & 1) == 0 && (reinterpret_cast<uintptr_t>(res) & 3) == 0;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < pairs;
         g += (long long)gridDim.x * blockDim.x) {
        const long long i = 2 * g;
        const bool two = i + 1 < count;
        unsigned long long a[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
        for (int t0 = 0; t0 < p.n; t0 += kCrtBatch) {
            unsigned int word[kCrtBatch];
#pragma unroll
            for (int u = 0; u < kCrtBatch; ++u) {
                word[u] = 0;
                if (t0 + u < p.n) {
                    const short* src = res + (long long)(t0 + u) * count + i;
                    if (vec) {
                        word[u] = __ldg(reinterpret_cast<const unsigned int*>(src));
                    } else {
                        word[u] = (unsigned short)src[0];
                        if (two) word[u] |= (unsigned int)(unsigned short)src[1] << 16;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kCrtBatch; ++u) {
                if (t0 + u >= p.n) break;
                const int m = p.m[t0 + u];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    int r = (int)(short)(word[u] >> (16 * e));
                    r += r < 0 ? m : 0;
                    const unsigned int ru = (unsigned int)r;
                    a[e][0] += (unsigned long long)ru * p.w[t0 + u][0];
                    a[e][1] += (unsigned long long)ru * p.w[t0 + u][1];
                    a[e][2] += (unsigned long long)ru * p.w[t0 + u][2];
                    a[e][3] += (unsigned long long)ru * p.w[t0 + u][3];
                }
            }
        }
        const i128 x0 = crt_reduce(a[0][0], a[0][1], a[0][2], a[0][3], p, M, half);
        longlong2* dst = reinterpret_cast<longlong2*>(out + 2 * i);
        dst[0] = make_longlong2((long long)(unsigned long long)(u128)x0, (long long)(x0 >> 64));
        if (two) {
            const i128 x1 = crt_reduce(a[1][0], a[1][1], a[1][2], a[1][3], p, M, half);
            dst[1] = make_longlong2((long long)(unsigned long long)(u128)x1, (long long)(x1 >> 64));
        }
    }
}

bool build_crt_params(const int* moduli, int n, CrtParams* c) {
    c->n = n;
    u128 M = 1;
    for (int t = 0; t < n; ++t) M *= (u128)moduli[t];
    for (int t = 0; t < n; ++t) {
        const int m = moduli[t];
        const u128 Mt = M / (u128)m;
        const int mt_mod = (int)(Mt % (u128)m);
        int inv = 0;
        for (int a = 1; a < m && !inv; ++a)
            if ((mt_mod * a) % m == 1) inv = a;
        if (!inv) return false;
        const u128 W = Mt * (u128)inv;  // < M
        c->m[t] = m;
        for (int k = 0; k < 4; ++k) c->w[t][k] = (unsigned int)(W >> (32 * k));
    }
    for (int k = 0; k < 4; ++k) c->M[k] = (unsigned int)(M >> (32 * k));
    c->M_lo = (unsigned long long)M;
    c->M_hi = (unsigned long long)(M >> 64);
    c->half_lo = (unsigned long long)(M / 2);
    c->half_hi = (unsigned long long)((M / 2) >> 64);
    c->M_as_double = (double)c->M_hi * 18446744073709551616.0 + (double)c->M_lo;
    return true;
}

// Number of FP4 products the residue scheme of modulus m needs (1, 3 or 4).
int products_of(int m) {
    awe_encoding_desc d;
    return awe_encoding_info(AWE_ENC_MOD_M, m, &d) == AWE_OK ? d.r : 1 << 20;
}

// The paper chooses, by an integer program over the per-modulus costs, the moduli with the fewest
// products whose product exceeds 2 K B^2 (Section 5.3).  Over the 22 built-in moduli this is a small
// knapsack: best[c] = largest sum of log2(m) reachable with exactly c products; the cheapest c that
// reaches the bound wins and the exact inequality is re-checked in integers.
int select_moduli(int in_bits, int64_t K, int* out) {
    const long double need = 1.0L + log2l((long double)K) + 2.0L * (long double)(in_bits - 1);
    constexpr int kMaxCost = 64;
    long double best[kMaxCost + 1];
    unsigned int pick[kMaxCost + 1];
    for (int c = 0; c <= kMaxCost; ++c) {
        best[c] = -1;
        pick[c] = 0;
    }
    best[0] = 0;
    for (int t = 0; t < kNumWideModuli; ++t) {
        const int cost = products_of(kWideModuli[t]);
        const long double lg = log2l((long double)kWideModuli[t]);
        for (int c = kMaxCost; c >= cost; --c)
            if (best[c - cost] >= 0 && best[c - cost] + lg > best[c]) {
                best[c] = best[c - cost] + lg;
                pick[c] = pick[c - cost] | (1u << t);
            }
    }
    for (int c = 1; c <= kMaxCost; ++c) {
        if (best[c] < need) continue;
        // exact check: prod(m) > 2 K (2^(in_bits-1) - 1)^2, all below 2^128
        u128 prod = 1;
        for (int t = 0; t < kNumWideModuli; ++t)
            if (pick[c] >> t & 1) prod *= (u128)kWideModuli[t];
        const u128 B = ((u128)1 << (in_bits - 1)) - 1;
        const u128 bound = (u128)2 * (u128)K * B;  // prod > bound * B, written without forming bound * B
        if (!(prod / B > bound || (prod / B == bound && prod % B != 0))) continue;
        int n = 0;
        for (int t = 0; t < kNumWideModuli; ++t)
            if (pick[c] >> t & 1) out[n++] = kWideModuli[t];
        return n;
    }
    return 0;
}

struct WideLayout {
    size_t res_a, res_b, res_c, planes, total;
};

bool wide_layout(int64_t M, int64_t N, int64_t K, WideLayout* w) {
    size_t planes = 0;
    for (int t = 0; t < kNumWideModuli; ++t) {
        const size_t b = awe_workspace_bytes(AWE_ENC_MOD_M, kWideModuli[t], M, N, K);
        if (!b) return false;
        planes = std::max(planes, b);
    }
    size_t off = 0;
    w->res_a = off;
    off += (size_t)round_up((int64_t)kNumWideModuli * M * K, 256);
    w->res_b = off;
    off += (size_t)round_up((int64_t)kNumWideModuli * K * N, 256);
    w->res_c = off;
    off += (size_t)round_up((int64_t)kNumWideModuli * M * N * 2, 256);
    w->planes = off;
    off += (size_t)round_up((int64_t)planes, 256);
    w->total = off;
    return true;
}

}  // namespace

extern "C" int awe_wide_moduli(int32_t* out, int capacity) {
    if (out)
        for (int t = 0; t < kNumWideModuli && t < capacity; ++t) out[t] = kWideModuli[t];
    return kNumWideModuli;
}

extern "C" size_t awe_wide_workspace_bytes(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    WideLayout w;
    return wide_layout(M, N, K, &w) ? w.total : 0;
}

static awe_status_t launch_residues(awe_handle_t h, const int64_t* X_dev, int64_t count, const int* moduli, int n,
                                    int8_t* res_dev, void* stream) {
    if (!h || !X_dev || !res_dev || count <= 0) return AWE_ERR_INVALID_ARG;
    if ((uintptr_t)X_dev % 16 || (uintptr_t)res_dev % 4) return AWE_ERR_ALIGNMENT;
    ResidueParams p = {};
    p.n = n;
    for (int t = 0; t < n; ++t) {
        const unsigned int m = (unsigned int)moduli[t];
        p.mf[t] = (float)m;
        p.inv_m[t] = 1.0f / (float)m;
        p.c1f[t] = (float)((1u << 14) % m);
        p.c2f[t] = (float)((1u << 28) % m);
        p.c3f[t] = (float)((1ull << 42) % m);
        p.lo[t] = -(float)(m / 2);
        p.hi[t] = (float)((m + 1) / 2) - 1.0f;
    }
    const long long groups = (count + 3) / 4;
    const unsigned blocks = (unsigned)std::min<long long>((groups + 255) / 256, (long long)h->sm_count * 16);
    wide_residues_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>((const long long*)X_dev, count, p, res_dev);
    if (cudaGetLastError() != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

extern "C" awe_status_t awe_wide_residues(awe_handle_t h, const int64_t* X_dev, int64_t count, int8_t* res_dev,
                                          void* stream) {
    return launch_residues(h, X_dev, count, kWideModuli, kNumWideModuli, res_dev, stream);
}

static awe_status_t launch_crt(awe_handle_t h, const int16_t* res_dev, int64_t count, const int* moduli, int n,
                               int64_t* out_dev, void* stream) {
    if (!h || !res_dev || !out_dev || count <= 0) return AWE_ERR_INVALID_ARG;
    if ((uintptr_t)res_dev % 2 || (uintptr_t)out_dev % 16) return AWE_ERR_ALIGNMENT;
    CrtParams c = {};
    if (!build_crt_params(moduli, n, &c)) return AWE_ERR_UNSUPPORTED;
    const unsigned blocks = (unsigned)std::min<long long>(((count + 1) / 2 + 255) / 256, (long long)h->sm_count * 16);
    wide_crt_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>((const short*)res_dev, count, c, (long long*)out_dev);
    if (cudaGetLastError() != cudaSuccess) return AWE_ERR_CUDA;
    h->launches += 1;
    return AWE_OK;
}

extern "C" awe_status_t awe_wide_crt(awe_handle_t h, const int16_t* res_dev, int64_t count, int64_t* out_dev,
                                     void* stream) {
    return launch_crt(h, res_dev, count, kWideModuli, kNumWideModuli, out_dev, stream);
}

extern "C" int awe_wide_select(int in_bits, int64_t K, int32_t* out, int capacity) {
    if (in_bits < 2 || in_bits > 54 || K <= 0) return 0;
    int sel[kMaxModuli];
    const int n = select_moduli(in_bits, K, sel);
    if (out)
        for (int t = 0; t < n && t < capacity; ++t) out[t] = sel[t];
    return n;
}

extern "C" awe_status_t awe_gemm_exact_wide(awe_handle_t h, const int64_t* A_dev, const int64_t* B_dev, int64_t M,
                                            int64_t N, int64_t K, int in_bits, int64_t* C_dev, void* workspace_dev,
                                            size_t workspace_bytes, void* stream) {
    if (!h || !A_dev || !B_dev || !C_dev || !workspace_dev || M <= 0 || N <= 0 || K <= 0) return AWE_ERR_INVALID_ARG;
    if (in_bits < 2 || in_bits > 54) return AWE_ERR_INVALID_ARG;
    // unique reconstruction: prod(m) > 2 K B^2 with B = 2^(in_bits-1) - 1  (Section 5.3); the cheapest
    // subset of the built-in moduli that satisfies it is used
    int sel[kMaxModuli];
    const int n_sel = select_moduli(in_bits, K, sel);
    if (n_sel == 0) return AWE_ERR_RANGE;
    WideLayout w;
    if (!wide_layout(M, N, K, &w)) return AWE_ERR_UNSUPPORTED;
    if (workspace_bytes < w.total) return AWE_ERR_WORKSPACE;
    if ((uintptr_t)workspace_dev % 256 || (uintptr_t)A_dev % 16 || (uintptr_t)B_dev % 16 || (uintptr_t)C_dev % 16)
        return AWE_ERR_ALIGNMENT;
    uint8_t* base = (uint8_t*)workspace_dev;
    int8_t* res_a = (int8_t*)(base + w.res_a);
    int8_t* res_b = (int8_t*)(base + w.res_b);
    int16_t* res_c = (int16_t*)(base + w.res_c);
    awe_status_t s;
    if ((s = launch_residues(h, A_dev, M * K, sel, n_sel, res_a, stream)) != AWE_OK) return s;
    if ((s = launch_residues(h, B_dev, K * N, sel, n_sel, res_b, stream)) != AWE_OK) return s;
    for (int t = 0; t < n_sel; ++t) {
        s = awe_gemm_exact(h, res_a + (size_t)t * M * K, AWE_I8, res_b + (size_t)t * K * N, AWE_I8, M, N, K,
                           AWE_ENC_MOD_M, sel[t], res_c + (size_t)t * M * N, AWE_C_RES_I16, base + w.planes,
                           w.total - w.planes, stream);
        if (s != AWE_OK) return s;
    }
    return launch_crt(h, res_c, M * N, sel, n_sel, C_dev, stream);
}

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
constexpr int kNumWideModuli = 22;
constexpr int kWideModuli[kNumWideModuli] = {7,  8,  9,  11, 13, 41, 43, 47, 53,  59,  61,
                                             67, 71, 73, 79, 83, 85, 89, 139, 149, 151, 157};

typedef unsigned __int128 u128;
typedef __int128 i128;

// 2^e mod m in the symmetric range, as a float.
constexpr float pow2_mod_symmetric(int e, int m) {
    int r = 1 % m;
    for (int i = 0; i < e; ++i) r = (2 * r) % m;
    return (float)(r > m / 2 ? r - m : r);
}

// Built-in modulus number T with the constants of its residue computation, all compile-time.
template <int T>
struct WideModulus {
    static constexpr int m = kWideModuli[T];
    static constexpr float mf = (float)m, inv_m = 1.0f / (float)m;
    static constexpr float c1 = pow2_mod_symmetric(14, m), c2 = pow2_mod_symmetric(28, m),
                           c3 = pow2_mod_symmetric(42, m);
};

struct ResidueParams {
    unsigned int mask;                // bit T: built-in modulus T is wanted
    long long offset[kNumWideModuli]; // its residues start at out + offset[T]
};

constexpr float kRoundMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds |v| < 2^22 to an integer held in the low mantissa bits

// x mod m for built-in modulus T, on the FP32 pipe.  f holds the four signed 14-bit limbs of x as floats
// (x = f0 + f1 2^14 + f2 2^28 + f3 2^42).  s = f0 + f1 c1 + f2 c2 + f3 c3 with c_k = 2^(14k) mod m taken
// in the symmetric range is an integer of magnitude below 2^14 (1 + 3 m / 2) < 2^22, hence exact;
// q = round(s / m) by one FMA with the rounding constant (the estimate s * (1/m) is off by less than
// 0.23 / m while every non-integer multiple of 1/m is at least 0.5 / m away from a rounding boundary, so
// q is the exact nearest integer, either neighbour on a tie); r = s - q m is then exact with
// |r| <= m / 2, which is the symmetric range except for r = +m/2 of an even modulus.  Returns
// r + 1.5 * 2^23 as bits: the low byte is r in two's complement.
template <int T>
__device__ __forceinline__ uint32_t symmetric_residue_bits(const float (&f)[4]) {
    typedef WideModulus<T> W;
    const float s = __fmaf_rn(f[3], W::c3, __fmaf_rn(f[2], W::c2, __fmaf_rn(f[1], W::c1, f[0])));
    const float q = __fadd_rn(__fmaf_rn(s, W::inv_m, kRoundMagic), -kRoundMagic);
    float r = __fmaf_rn(-q, W::mf, s);
    if (W::m % 2 == 0) r = (r == (float)(W::m / 2)) ? -r : r;
    return __float_as_uint(__fadd_rn(r, kRoundMagic));
}

// Signed 14-bit limbs of x (|x| < 2^56) as floats: a limb l < 2^14 placed in the mantissa of 2^23 reads
// as 2^23 + l, and one FMA with +-1 removes the offset and applies the sign of x.
__device__ __forceinline__ void split14_signed(long long x, float (&f)[4]) {
    const unsigned long long ax = x < 0 ? (unsigned long long)(-x) : (unsigned long long)x;
    const float sgn = x < 0 ? -1.0f : 1.0f, off = x < 0 ? 8388608.0f : -8388608.0f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t limb = (uint32_t)(ax >> (14 * k)) & 0x3FFFu;
        f[k] = __fmaf_rn(__uint_as_float(0x4B000000u | limb), sgn, off);
    }
}

constexpr int kResPerThread = 8;  // consecutive elements per thread: one 8-byte store per modulus

template <int T>
__device__ __forceinline__ void residues_of_group(const float (&f)[kResPerThread][4], const ResidueParams& p,
                                                  int8_t* out, long long i0, long long count, bool full) {
    if (p.mask >> T & 1u) {  // the same for every thread
        uint32_t word[kResPerThread / 4];
#pragma unroll
        for (int w = 0; w < kResPerThread / 4; ++w) {
            const uint32_t b0 = symmetric_residue_bits<T>(f[4 * w]), b1 = symmetric_residue_bits<T>(f[4 * w + 1]);
            const uint32_t b2 = symmetric_residue_bits<T>(f[4 * w + 2]), b3 = symmetric_residue_bits<T>(f[4 * w + 3]);
            word[w] = __byte_perm(__byte_perm(b0, b1, 0x0040), __byte_perm(b2, b3, 0x0040), 0x5410);
        }
        int8_t* dst = out + p.offset[T] + i0;
        if (full) {
            *reinterpret_cast<uint2*>(dst) = make_uint2(word[0], word[1]);
        } else {
            for (int j = 0; j < kResPerThread; ++j)
                if (i0 + j < count) dst[j] = (int8_t)(word[j / 4] >> (8 * (j % 4)));
        }
    }
    if constexpr (T + 1 < kNumWideModuli) residues_of_group<T + 1>(f, p, out, i0, count, full);
}

// X: `count` 64-bit integers; out[offset[T] + i] = symmetric residue of X[i] modulo built-in modulus T
// for every T in the mask.  A thread takes 8 consecutive elements so every store is an 8-byte word and a
// warp writes 256 contiguous bytes per modulus; the loop over the moduli is unrolled at compile time, so
// their constants are immediates.  `vec`: every modulus' array starts on an 8-byte boundary.
__global__ void __launch_bounds__(256)
wide_residues_kernel(const long long* __restrict__ X, long long count, const __grid_constant__ ResidueParams p,
                     int8_t* __restrict__ out, int vec) {
    const long long groups = (count + kResPerThread - 1) / kResPerThread;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < groups;
         g += (long long)gridDim.x * blockDim.x) {
        const long long i0 = g * kResPerThread;
        long long x[kResPerThread];
        if (i0 + kResPerThread <= count) {
#pragma unroll
            for (int j = 0; j < kResPerThread / 2; ++j) {
                const longlong2 a = __ldg(reinterpret_cast<const longlong2*>(X + i0) + j);
                x[2 * j] = a.x;
                x[2 * j + 1] = a.y;
            }
        } else {
            for (int j = 0; j < kResPerThread; ++j) x[j] = i0 + j < count ? X[i0 + j] : 0;
        }
        float f[kResPerThread][4];  // signed 14-bit limbs of the elements
#pragma unroll
        for (int j = 0; j < kResPerThread; ++j) split14_signed(x[j], f[j]);
        residues_of_group<0>(f, p, out, i0, count, vec && i0 + kResPerThread <= count);
    }
}

struct CrtParams {
    unsigned int mask;                  // bit T: built-in modulus T takes part
    long long offset[kNumWideModuli];   // its residues start at res + offset[T] (elements)
    int w[kNumWideModuli][4];           // W_T = (M/m_T) ((M/m_T)^-1 mod m_T) < 2^123 in four 31-bit limbs
    int M[4];                           // M = prod m_T in 31-bit limbs
    unsigned long long M_lo, M_hi, half_lo, half_hi;
    double inv_M;                       // 1 / M rounded to double
};

// res[offset[T] + i]: residues of the unknown integers modulo m_T (any representative that fits 16 bits;
// the products deliver the symmetric one).  The integer with -M/2 < x <= M/2 is x = sum_T r_T W_T mod M
// (textbook CRT).  The sum is formed limb by limb with signed 32 x 32 -> 64-bit multiply-adds (W_T in
// 31-bit limbs so that they are positive as signed words; 22 terms below 2^46 each, no carries needed),
// the quotient by M (|q| < 2^20) is estimated in double precision (one multiplication by 1/M: off by at
// most one), q M is subtracted limb by limb, carries are propagated once, and at most two corrections
// fix the estimate.  (The same sums as exact FP32 FMAs over 12-bit limbs of W_T, 11 per residue instead
// of 4 multiply-adds, were measured slower: 1.43 against 1.16 ms for 8192 x 8192 results.)
__device__ __forceinline__ i128 crt_reduce(const long long (&a)[4], const CrtParams& p, i128 M, i128 half) {
    const double two31 = 2147483648.0;
    const double xd = (((double)a[3] * two31 + (double)a[2]) * two31 + (double)a[1]) * two31 + (double)a[0];
    const long long q = (long long)floor(xd * p.inv_M);
    // d_k = a_k - q M_k (|d_k| < 2^52), then x - q M = sum_k d_k 2^(31 k) with signed carries
    long long c = a[0] - q * (long long)p.M[0];
    const unsigned long long r0 = (unsigned long long)c & 0x7FFFFFFFull;
    c = (c >> 31) + a[1] - q * (long long)p.M[1];
    const unsigned long long r1 = (unsigned long long)c & 0x7FFFFFFFull;
    c = (c >> 31) + a[2] - q * (long long)p.M[2];
    const unsigned long long r2 = (unsigned long long)c & 0x7FFFFFFFull;
    c = (c >> 31) + a[3] - q * (long long)p.M[3];  // top limb: signed and small, since |x - q M| < 2 M < 2^124
    i128 x = (i128)c * ((i128)1 << 93) + (i128)(((u128)r2 << 62) | ((u128)r1 << 31) | (u128)r0);
    if (x < 0) x += M;
    if (x >= M) x -= M;
    if (x > half) x -= M;
    return x;
}

// The two residues (elements i and i + 1) of built-in modulus T as one word; 0 where T takes no part.
template <int T>
__device__ __forceinline__ void crt_load(const CrtParams& p, const short* __restrict__ res, long long i, bool vec,
                                         bool two, unsigned int (&word)[kNumWideModuli]) {
    word[T] = 0;
    if (p.mask >> T & 1u) {
        const short* src = res + p.offset[T] + i;
        if (vec) {
            word[T] = __ldg(reinterpret_cast<const unsigned int*>(src));
        } else {
            word[T] = (unsigned short)src[0];
            if (two) word[T] |= (unsigned int)(unsigned short)src[1] << 16;
        }
    }
    if constexpr (T + 1 < kNumWideModuli) crt_load<T + 1>(p, res, i, vec, two, word);
}

template <int T>
__device__ __forceinline__ void crt_accumulate(const CrtParams& p, const unsigned int (&word)[kNumWideModuli],
                                               long long (&a)[2][4]) {
    if (p.mask >> T & 1u) {
        const int r0 = (int)(word[T] << 16) >> 16, r1 = (int)word[T] >> 16;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            a[0][k] += (long long)r0 * (long long)p.w[T][k];
            a[1][k] += (long long)r1 * (long long)p.w[T][k];
        }
    }
    if constexpr (T + 1 < kNumWideModuli) crt_accumulate<T + 1>(p, word, a);
}

// A thread takes two neighbouring elements: one 4-byte load per modulus (a warp reads whole 128-byte
// lines), the loads of all moduli in flight together, the loop over the moduli unrolled at compile time
// (the limbs of W_T are then operands straight from the parameter bank), and the two 128-bit results
// leave as one 32-byte sector.
__global__ void __launch_bounds__(256)
wide_crt_kernel(const short* __restrict__ res, long long count, const __grid_constant__ CrtParams p,
                long long* __restrict__ out, int vec_ok) {
    const i128 M = (i128)(((u128)p.M_hi << 64) | p.M_lo);
    const i128 half = (i128)(((u128)p.half_hi << 64) | p.half_lo);
    const long long pairs = (count + 1) / 2;
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < pairs;
         g += (long long)gridDim.x * blockDim.x) {
        const long long i = 2 * g;
        const bool two = i + 1 < count;
        unsigned int word[kNumWideModuli];
        crt_load<0>(p, res, i, vec_ok != 0, two, word);
        long long a[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
        crt_accumulate<0>(p, word, a);
        const i128 x0 = crt_reduce(a[0], p, M, half);
        longlong2* dst = reinterpret_cast<longlong2*>(out + 2 * i);
        dst[0] = make_longlong2((long long)(unsigned long long)(u128)x0, (long long)(x0 >> 64));
        if (two) {
            const i128 x1 = crt_reduce(a[1], p, M, half);
            dst[1] = make_longlong2((long long)(unsigned long long)(u128)x1, (long long)(x1 >> 64));
        }
    }
}

// moduli[t] (each one of the built-in set, no repeats) with its residues at res + t * count.
bool build_crt_params(const int* moduli, int n, long long count, CrtParams* c) {
    u128 M = 1;
    for (int t = 0; t < n; ++t) M *= (u128)moduli[t];
    for (int t = 0; t < n; ++t) {
        const int m = moduli[t];
        int T = 0;
        while (T < kNumWideModuli && kWideModuli[T] != m) ++T;
        if (T == kNumWideModuli || (c->mask >> T & 1u)) return false;
        const u128 Mt = M / (u128)m;
        const int mt_mod = (int)(Mt % (u128)m);
        int inv = 0;
        for (int a = 1; a < m && !inv; ++a)
            if ((mt_mod * a) % m == 1) inv = a;
        if (!inv) return false;
        const u128 W = Mt * (u128)inv;  // < M
        c->mask |= 1u << T;
        c->offset[T] = (long long)t * count;
        for (int k = 0; k < 4; ++k) c->w[T][k] = (int)((W >> (31 * k)) & 0x7FFFFFFFu);
    }
    for (int k = 0; k < 4; ++k) c->M[k] = (int)((M >> (31 * k)) & 0x7FFFFFFFu);
    c->M_lo = (unsigned long long)M;
    c->M_hi = (unsigned long long)(M >> 64);
    c->half_lo = (unsigned long long)(M / 2);
    c->half_hi = (unsigned long long)((M / 2) >> 64);
    c->inv_M = 1.0 / ((double)c->M_hi * 18446744073709551616.0 + (double)c->M_lo);
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
    // residues of moduli[t] go to res_dev + t * count; every modulus must be one of the built-in set
    ResidueParams p = {};
    for (int t = 0; t < n; ++t) {
        int T = 0;
        while (T < kNumWideModuli && kWideModuli[T] != moduli[t]) ++T;
        if (T == kNumWideModuli || (p.mask >> T & 1u)) return AWE_ERR_UNSUPPORTED;
        p.mask |= 1u << T;
        p.offset[T] = (long long)t * count;
    }
    const long long groups = (count + kResPerThread - 1) / kResPerThread;
    const unsigned blocks = (unsigned)std::min<long long>((groups + 255) / 256, (long long)h->sm_count * 16);
    const int vec = (count % 8 == 0) && ((uintptr_t)res_dev % 8 == 0);
    wide_residues_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>((const long long*)X_dev, count, p, res_dev, vec);
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
    if (!build_crt_params(moduli, n, count, &c)) return AWE_ERR_UNSUPPORTED;
    const unsigned blocks = (unsigned)std::min<long long>(((count + 1) / 2 + 255) / 256, (long long)h->sm_count * 16);
    // every modulus' array starts on a 4-byte boundary
    const int vec_ok = (count & 1) == 0 && ((uintptr_t)res_dev & 3) == 0;
    wide_crt_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>((const short*)res_dev, count, c, (long long*)out_dev,
                                                             vec_ok);
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

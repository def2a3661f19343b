// Internal declarations shared by the translation units of the AWE library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "awe.h"

namespace awe {

constexpr int kMaxLimbs = 4;

// One configuration record (Definition 4.1): weights, planes per product, integer
// reconstruction coefficients, denominator 2^log2D, optional modulus (Section 5.3).
struct Scheme {
    int p = 0, q = 0, r = 0;
    int w[kMaxLimbs] = {0}, v[kMaxLimbs] = {0};
    int alpha[AWE_MAX_PRODUCTS][kMaxLimbs] = {{0}};
    int beta[AWE_MAX_PRODUCTS][kMaxLimbs] = {{0}};
    int ell[AWE_MAX_PRODUCTS] = {0};
    int log2D = 0;
    int modulus = 0;
    int a_lo = -128, a_hi = 127, b_lo = -128, b_hi = 127;
};

// Stored planes of one side and the per-byte table derived from the record.
struct SideTable {
    int n_planes = 0;
    int planes[AWE_MAX_PLANES][kMaxLimbs] = {{0}};
    int index_of_product[AWE_MAX_PRODUCTS] = {0};
    int index2_of_product[AWE_MAX_PRODUCTS];  // second stored plane whose sum with the first is multiplied, or -1
    SideTable() { for (int& x : index2_of_product) x = -1; }
    int bits[AWE_MAX_PLANES] = {4, 4, 4, 4, 4, 4, 4, 4};  // storage width: 4 = E2M1 nibble, 8 = E4M3 byte
    int c = 0;       // largest |plane value| over the input range
    int entries = 0; // 256 (index: raw byte) or 4096 (index: low 12 bits of a 16-bit element)
    std::vector<int8_t> value;  // entries x AWE_MAX_PLANES plane values
    std::vector<uint64_t> lut;  // entries words: E2M1 code of plane j in the low nibble of byte j
};

// Builds (and caches) scheme + tables; returns false if the encoding/modulus is not available.
bool get_scheme(int enc, int modulus, Scheme* out);
bool get_side_table(int enc, int modulus, awe_side_t side, awe_in_dtype_t dt, const SideTable** out);
awe_in_dtype_t natural_dtype(int enc, awe_side_t side);

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline int64_t plane_pitch_bytes(int64_t K) { return round_up(K, 256) / 2; }
// Storage of one input element in half-bytes: 4 for 16-bit elements, 1 for packed 4-bit, else 2.
inline bool is_16bit(awe_in_dtype_t dt) { return dt == AWE_I16 || dt == AWE_I9_IN_I16; }
inline int64_t in_elem_nibbles(awe_in_dtype_t dt) { return is_16bit(dt) ? 4 : (dt == AWE_I4_PACKED ? 1 : 2); }
inline int64_t in_bytes(awe_in_dtype_t dt, int64_t count) { return (count * in_elem_nibbles(dt) + 1) / 2; }
// Packed 4-bit inputs share the table of the one-value-per-byte container.
inline awe_in_dtype_t table_dtype(awe_in_dtype_t dt) { return dt == AWE_I4_PACKED ? AWE_I4_IN_I8 : dt; }
// Size of one row of all stored planes of a side, in units of the E2M1 pitch.
// The epilogue keeps sum_k l_k P_k = D*C modulo 2^32 and shifts by log2 D afterwards (Definition 4.1),
// so 32-bit running sums need |D*C| <= D max|a| max|b| K below 2^31.  When not even one 256-element
// K block satisfies that, the products run through the kernel with 64-bit sums instead.
inline int64_t input_bound(const awe_encoding_desc& d) {
    const int64_t amax = d.a_lo < 0 && -(int64_t)d.a_lo > d.a_hi ? -(int64_t)d.a_lo : d.a_hi;
    const int64_t bmax = d.b_lo < 0 && -(int64_t)d.b_lo > d.b_hi ? -(int64_t)d.b_lo : d.b_hi;
    return amax * bmax;
}
inline bool needs_wide_sums(const awe_encoding_desc& d) {
    return d.modulus == 0 && ((int64_t)1 << 30) / (input_bound(d) << d.log2D) < 256;
}
// int32 output: the result itself must fit, and so must D*C wherever the sums are 32 bits wide.
inline bool i32_output_fits(const awe_encoding_desc& d, int64_t K) {
    const __int128 c = (__int128)input_bound(d) * K;
    return (needs_wide_sums(d) ? c : c << d.log2D) < ((__int128)1 << 31);
}
inline int plane_units(const int32_t* bits, int n_planes) {
    int u = 0;
    for (int j = 0; j < n_planes; ++j) u += bits[j] / 4;
    return u;
}

}  // namespace awe

struct awe_ctx {
    int device = 0;
    int sm_count = 0;
    unsigned int* status_dev = nullptr;  // [0] = status, [1] = site, [2..5] = clock probe of the last GEMM launch
    uint64_t* lut_arena_dev = nullptr;   // lut_slots tables of 256 x u64
    int lut_slots = 0;                   // capacity of that arena
    uint64_t* lut16_arena_dev = nullptr; // kLut16Slots tables of 4096 x u64 (16-bit inputs)
    struct Lut16Slot {
        int enc, side;
    };
    std::vector<Lut16Slot> slots16;
    struct LutSlot {
        int enc, modulus, side, dt;
    };
    std::vector<LutSlot> slots;
    int64_t launches = 0;
    void* encode_tiled = nullptr;  // cuTensorMapEncodeTiled, resolved through the runtime
    // copy engines of the host-buffer entry point: one stream per direction and the events that
    // order them against the caller's stream (created on first use)
    static constexpr int kMaxHostChunks = 16;   // row chunks of A and C
    static constexpr int kMaxHostColBlocks = 8;  // column blocks of B and C
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_b = nullptr, ev_done = nullptr;
    cudaEvent_t ev_a[kMaxHostChunks] = {nullptr}, ev_bcol[kMaxHostColBlocks] = {nullptr};
    cudaEvent_t ev_c[kMaxHostChunks * kMaxHostColBlocks] = {nullptr};
    bool smem_attr_set[32] = {false};  // dynamic shared-memory limit raised (per kernel, this device)
};

namespace awe {
// The stored planes of an operand seen as a window of rows [row0, row0 + R) inside a plane set whose
// planes are plane_rows rows apart (the whole set when row0 = 0 and plane_rows = R).  Lets the
// host-buffer path encode an operand chunk by chunk into one plane set and multiply any row range of it.
struct PlaneWindow {
    const void* base;    // start of the whole plane set
    int64_t plane_rows;  // rows per plane of the whole set
    int64_t row0;        // first row of the window
};
awe_status_t encode_window(awe_ctx* h, int enc, int modulus, awe_side_t side, const void* X_dev, awe_in_dtype_t dt,
                           awe_layout_t layout, int64_t R, int64_t K, int64_t ld, PlaneWindow win, void* stream);
awe_status_t gemm_planes_window(awe_ctx* h, int enc, int modulus, PlaneWindow a, PlaneWindow b, int64_t M, int64_t N,
                                int64_t K, void* C_dev, awe_out_dtype_t out_dt, int64_t ldc, int64_t k_chunk,
                                void* stream);
// Table arena of a handle: room for both sides of every modulus 2..169 and of every exact
// encoding in each input container, so that no table ever has to be evicted.
constexpr int kLutSlots = 512;
// The allocation-free context keeps its tables inside the built-in array and has room for fewer.
constexpr int kStaticLutSlots = 96;
constexpr int kLut16Slots = 4;
constexpr int kStatusWords = 8;
// Device pointer of the 256-entry u64 table for (enc, modulus, side, dt); uploads on first use.
awe_status_t device_lut(awe_ctx* h, int enc, int modulus, awe_side_t side, awe_in_dtype_t dt,
                        cudaStream_t stream, const uint64_t** out);
}  // namespace awe

/* awe.h -- C ABI of the B200 (sm_100a) library for error-free integer matrix products
 * computed as a few FP4 (E2M1) tensor-core GEMMs under Adaptive Weight Encoding (AWE).
 *
 * What the library computes is the run-time procedure of the paper (Algorithm 1):
 *   1. every entry of A and of B is decomposed into limbs by table lookup and the stored
 *      planes (linear combinations of limbs, every value in S = {0,+-1,+-2,+-3,+-4,+-6,+-8,+-12})
 *      are written as packed E2M1 (awe_encode);
 *   2. for each product k = 1..r, P_k = plane alpha_k of A times plane beta_k of B on the FP4
 *      tensor cores with FP32 accumulation, the reduction dimension cut into segments short
 *      enough (Section 3.4, K*) that every partial sum is an integer below 2^24 and exact;
 *      products of equal coefficient share an accumulator where that keeps the sum exact (n_g
 *      of Section 3.4), and the record of Appendix A that mixes formats runs two of its three
 *      products on E4M3 planes (FP8 tensor cores, same accumulation rule);
 *   3. C = (sum_k l_k P_k) / D in integers, D a power of two (Definition 4.1), or the same sum
 *      reduced mod m for the residue form (Section 5.3)
 *   (steps 2 and 3: awe_gemm_planes; all three: awe_gemm_exact).
 *
 * Conventions that hold for every entry point unless its comment says otherwise:
 *   - Pointers named *_dev are DEVICE pointers into memory the caller owns (cudaMalloc'd or a
 *     framework tensor); pointers named *_host are HOST pointers.  The library never frees or
 *     keeps a caller pointer past the call's enqueued work.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Device
 *     work is enqueued on it and the call returns without waiting, except where stated.
 *   - No entry point allocates device memory per call; scratch is caller-provided
 *     (awe_workspace_bytes).  A handle owns a small device status word and the encode tables.
 *   - Errors the host can see (bad argument, unsupported encoding, misalignment, short
 *     workspace, result range) are returned before anything is enqueued.  Conditions only the
 *     device can see (a bounded wait inside a kernel ran out) are recorded in the handle's
 *     status word and reported by awe_last_device_status.
 *   - There is no CPU fallback: without a CUDA device awe_create fails with AWE_ERR_CUDA.
 *   - The first use of an encoding on a handle uploads its tables and waits for that copy; from then
 *     on awe_encode, awe_gemm_planes and awe_gemm_exact only enqueue kernels on `stream`, so a
 *     warmed-up call can be captured in a CUDA graph and replayed (the tests do this).
 *   - One handle serves one device; calls on one handle must not run concurrently from
 *     several host threads.
 */
#ifndef AWE_H_
#define AWE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct awe_ctx* awe_handle_t;

typedef enum {
    AWE_OK = 0,
    AWE_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, unknown enum value            */
    AWE_ERR_UNSUPPORTED = 2, /* encoding/modulus/dtype combination the library does not have   */
    AWE_ERR_WORKSPACE = 3,   /* caller-provided scratch is too small                           */
    AWE_ERR_ALIGNMENT = 4,   /* a pointer or leading dimension misses its alignment            */
    AWE_ERR_RANGE = 5,       /* the exact result cannot fit the requested output type          */
    AWE_ERR_CUDA = 6,        /* a CUDA runtime or driver call failed                           */
    AWE_ERR_TIMEOUT = 7      /* a bounded wait inside a kernel expired (device status word)    */
} awe_status_t;

/* Encodings (configuration records of Algorithm 1). */
typedef enum {
    AWE_ENC_INT8_AWE6 = 1,      /* INT8xINT8, 6 products, w = v = (1,29,37)   (Section 4.3, Appendix A) */
    AWE_ENC_INT8_BASE13_9 = 2,  /* INT8xINT8, 9 products, weights (1,13,169)  (prior work, Section 1)  */
    AWE_ENC_INT4xINT8_AWE4 = 3, /* INT4xINT8, 4 products, D = 2               (Appendix A)             */
    AWE_ENC_MOD_M = 4,          /* residue form mod `modulus`, 1/3/4 products (Section 5.3)            */
    AWE_ENC_INT8_AWE6_ALT = 5,  /* INT8xINT8, 6 products, w = v = (1,11,39)   (Section 4.3)            */
    AWE_ENC_TERNARY_INT8_3 = 6, /* {0,+-1}xINT8, 3 products: one limb against the three base-13 limbs
                                   (Section 6.2), K* = 2,097,152                                       */
    AWE_ENC_INT4xINT4_3 = 7,    /* INT4xINT4, 3 products (count from Section 5.2; the encoding is not
                                   printed: planes a0, a1, a0-a1 with weights (1,3))                  */
    AWE_ENC_FP16SIG_AWE12 = 8,  /* width-12 integers (FP16 significands with sign, |x| <= 2047; the
                                   table also covers -2048), 12 products, w = v = (1,9,71,639), D = 2
                                   (Appendix A).  16-bit inputs (AWE_I16); 64-bit reconstruction.     */
    AWE_ENC_INT8_MIXED_FP8_3 = 9, /* INT8xINT8 with 2 FP8 products and 1 FP4 product (Appendix A):
                                   x = 13 h + 5 eps, planes h and h + eps stored as E4M3 bytes
                                   (|.| <= 14), eps in S (|eps| <= 8) as E2M1;
                                   xy = 104 hh' + 65 (h+eps)(h'+eps') - 40 eps eps', K* = 85,598.     */
    AWE_ENC_FP8SIG_3 = 10,      /* FP8 (E4M3) significands with sign, |x| <= 15 (the table also covers
                                   -16), 3 products: the Karatsuba-type step on two limbs (Section 6.1;
                                   the weights are not printed: w = v = (1,4), planes a0, a1, a0-a1,
                                   xy = 5 a0b0 + 20 a1b1 - 4 (a0-a1)(b0-b1)).  Inputs AWE_I5_IN_I8.    */
    AWE_ENC_BF16SIG_8 = 11,     /* BF16 significands with sign (width 9, |x| <= 255; the table also
                                   covers -256), 8 products (count from Section 6.2's table; the record
                                   is not printed): w = v = (4,9,61), planes a0, a1, a2, a0+a1, one
                                   Karatsuba-type step on the pair (a0, a1),
                                   xy = -20 a0b0 + 45 a1b1 + 3721 a2b2 + 36 (a0+a1)(b0+b1)
                                        + 244 (a0b2 + a2b0) + 549 (a1b2 + a2b1).  Inputs AWE_I9_IN_I16. */
    AWE_ENC_INT8_AWE6_DERIVED = 12 /* the record of AWE_ENC_INT8_AWE6 with only its three limb planes per side
                                   stored; the planes a_i + a_j of products 4..6 are formed inside the
                                   product kernel, in shared memory, from the limb tiles (the alternative
                                   Section 6.1 weighs when it speaks of the cost of producing planes).
                                   Half the plane bytes, same result; kept as a measured comparison.   */
} awe_encoding_t;

typedef enum {
    AWE_I8 = 0,      /* one signed 8-bit value per byte                                          */
    AWE_I4_IN_I8 = 1, /* one signed 4-bit value per byte; only the low nibble is read (sign-extended) */
    AWE_T2_IN_I8 = 2, /* one ternary value -1, 0 or +1 per byte; any other byte is read as 0         */
    AWE_I16 = 3,      /* one signed 12-bit value per 16-bit element; only the low 12 bits are read
                         (sign-extended).  Leading dimensions stay in elements.                      */
    AWE_I4_PACKED = 4, /* two signed 4-bit values per byte: element e of the row-major array sits in
                         byte e/2, the even one in the low nibble.  Leading dimensions stay in
                         elements and must be even (every row starts on a byte boundary).            */
    AWE_I5_IN_I8 = 5, /* one signed 5-bit value per byte; only the low 5 bits are read (sign-extended) */
    AWE_I9_IN_I16 = 6 /* one signed 9-bit value per 16-bit element; only the low 9 bits are read
                         (sign-extended).  Leading dimensions stay in elements.                      */
} awe_in_dtype_t;

typedef enum {
    AWE_C_I32 = 0,     /* exact product, int32 (rejected with AWE_ERR_RANGE if it might not fit) */
    AWE_C_I64 = 1,     /* exact product, int64                                                   */
    AWE_C_RES_I16 = 2, /* residue in [-floor(m/2), ceil(m/2)-1], int16 (AWE_ENC_MOD_M only)      */
    AWE_C_RES_I32 = 3  /* same residue, int32                                                    */
} awe_out_dtype_t;

typedef enum { AWE_SIDE_A = 0, AWE_SIDE_B = 1 } awe_side_t;

/* How the operand handed to awe_encode is laid out.  R is M for side A and N for side B. */
typedef enum {
    AWE_ROWMAJOR_RxK = 0, /* element (row r, reduction index k) at X[r*ld + k]  (A as M x K)     */
    AWE_ROWMAJOR_KxR = 1  /* element (r, k) at X[k*ld + r]                      (B as K x N)     */
} awe_layout_t;

#define AWE_MAX_PRODUCTS 16
#define AWE_MAX_PLANES 8

/* Host-side description of one configuration record (Definition 4.1 / Algorithm 1). */
typedef struct {
    int32_t r;                      /* number of products = number of FP4 GEMMs                  */
    int32_t n_planes_a, n_planes_b; /* distinct stored planes per side                           */
    int32_t ia[AWE_MAX_PRODUCTS];   /* product k multiplies stored plane ia[k] of A ...          */
    int32_t ib[AWE_MAX_PRODUCTS];   /* ... by stored plane ib[k] of B                            */
    int32_t ell[AWE_MAX_PRODUCTS];  /* integer reconstruction coefficients l_k                   */
    int32_t log2D;                  /* C = (sum l_k P_k) >> log2D                                */
    int32_t modulus;                /* 0 for the exact encodings                                 */
    int32_t c_a, c_b;               /* largest |stored plane value| per side (Section 3.4)       */
    int64_t k_star;                 /* floor(2^24 / (c_a c_b))                                   */
    int32_t a_lo, a_hi, b_lo, b_hi; /* input value range each side's table covers                */
    int32_t plane_bits_a[AWE_MAX_PLANES]; /* storage width of each stored plane: 4 (E2M1) or 8 (E4M3) */
    int32_t plane_bits_b[AWE_MAX_PLANES];
    int32_t fp8[AWE_MAX_PRODUCTS];  /* 1 if product k multiplies E4M3 planes (an FP8 GEMM), else 0 */
    int32_t ia2[AWE_MAX_PRODUCTS];  /* -1, or a second stored plane of A: product k multiplies the sum of */
    int32_t ib2[AWE_MAX_PRODUCTS];  /* planes ia[k] and ia2[k] (ib[k] and ib2[k]), formed in the kernel    */
} awe_encoding_desc;

/* Create / destroy a handle bound to CUDA device `device`.  awe_create makes that device
 * current, allocates the handle's status word and table arena (about 1 MB, once: room for the
 * tables of 512 (encoding, modulus, side, container) combinations, more than the library has) and
 * fails with AWE_ERR_CUDA if there is no usable sm_100 device.  (No counterpart in the paper.) */
awe_status_t awe_create(awe_handle_t* out, int device);
awe_status_t awe_destroy(awe_handle_t h);

/* Configuration record of an encoding (Definition 4.1; Appendix A; Section 5.3 for MOD_M, where
 * `modulus` in [2,169] selects the scheme and must be 0 otherwise).  Host only, needs no GPU.
 * AWE_ERR_UNSUPPORTED if no scheme exists for the modulus. */
awe_status_t awe_encoding_info(int enc, int modulus, awe_encoding_desc* out);

/* Decomposition table of one side (first two loops of Algorithm 1), host only: for every
 * raw input byte b (index b & 0xFF, interpreted per `dt`) the n_planes stored plane values,
 * lut_host[256 * n_planes], row b; for AWE_I16 the index is the low 12 bits of the element and the
 * table has 4096 rows.  Used to compare the table against an independent one. */
awe_status_t awe_encoding_lut(int enc, int modulus, awe_side_t side, awe_in_dtype_t dt, int8_t* lut_host);

/* Bytes of the packed-plane buffer of one operand: n_planes x R x pitch, pitch =
 * round_up(K,256)/2 bytes (E2M1, two values per byte, even k in the low nibble, zero padded
 * along K).  Planes stored as E4M3 (AWE_ENC_INT8_MIXED_FP8_3: planes 0 and 1) take one byte per
 * value, i.e. rows of 2 x pitch bytes; plane j starts where plane j-1 ends.  0 on invalid
 * arguments. */
size_t awe_planes_bytes(int enc, int modulus, awe_side_t side, int64_t R, int64_t K);

/* Bytes of scratch awe_gemm_exact needs (planes of A, then planes of B, each 256-B aligned). */
size_t awe_workspace_bytes(int enc, int modulus, int64_t M, int64_t N, int64_t K);

/* Extra device scratch awe_gemm_exact_host needs in addition to awe_workspace_bytes: room for
 * device copies of A, B and C. */
size_t awe_host_staging_bytes(int enc, int modulus, int64_t M, int64_t N, int64_t K, awe_out_dtype_t out_dt);

/* Encode one operand (Algorithm 1, first two loops): table lookup per value, plane formation,
 * E2M1 packing (E4M3 bytes for the FP8 planes of AWE_ENC_INT8_MIXED_FP8_3).  X_dev: R x K integers
 * laid out per `layout` with leading dimension ld (elements).  planes_dev: awe_planes_bytes bytes,
 * 256-B aligned.  Any ld and any alignment of X_dev are accepted (16-B aligned X_dev and
 * ld % 16 == 0 take the vectorised path); AWE_I4_PACKED needs an even ld (AWE_ERR_INVALID_ARG
 * otherwise) and vectorises with ld % 32 == 0 (R x K layout) or ld % 4 == 0 (K x R layout).
 * AWE_ERR_UNSUPPORTED if the encoding has no table for `dt` on this side. */
awe_status_t awe_encode(awe_handle_t h, int enc, int modulus, awe_side_t side, const void* X_dev,
                        awe_in_dtype_t dt, awe_layout_t layout, int64_t R, int64_t K, int64_t ld,
                        void* planes_dev, void* stream);

/* Products and reconstruction (Algorithm 1, third loop and last step; Section 3.4 for the
 * segmentation of K; Section 5.3 for the residue form) on planes written by awe_encode.
 * C_dev: M x N row-major with leading dimension ldc (elements of the output type), aligned to its
 * element size (16-B aligned rows, i.e. C_dev % 16 == 0 and ldc*sizeof(elem) % 16 == 0, take
 * the vector-store path).  k_chunk = 0 lets the library choose the segment length
 * (<= K* and a multiple of 256); a positive multiple of 256 forces it (testing); a forced length
 * above K* (above a quarter of K* for the residue form) would break exactness and is AWE_ERR_RANGE.
 * AWE_C_I32 needs D max|a| max|b| K < 2^31 (the sums are formed before the shift by log2 D),
 * AWE_ERR_RANGE otherwise. */
awe_status_t awe_gemm_planes(awe_handle_t h, int enc, int modulus, const void* planesA_dev,
                             const void* planesB_dev, int64_t M, int64_t N, int64_t K, void* C_dev,
                             awe_out_dtype_t out_dt, int64_t ldc, int64_t k_chunk, void* stream);

/* The whole of Algorithm 1: C = A.B exactly (or C mod m).  A_dev: M x K row-major (ld = K),
 * B_dev: K x N row-major (ld = N), C_dev: M x N row-major (ld = N).  workspace_dev: at least
 * awe_workspace_bytes bytes, 256-B aligned; its contents are overwritten.  A packed 4-bit operand
 * (AWE_I4_PACKED) needs an even K (as A) or an even N (as B). */
awe_status_t awe_gemm_exact(awe_handle_t h, const void* A_dev, awe_in_dtype_t a_dt, const void* B_dev,
                            awe_in_dtype_t b_dt, int64_t M, int64_t N, int64_t K, int enc, int modulus,
                            void* C_dev, awe_out_dtype_t out_dt, void* workspace_dev, size_t workspace_bytes,
                            void* stream);

/* Same product with HOST operands and result: copies A_host and B_host to the device, runs
 * awe_gemm_exact, copies C back to C_host and waits for the stream, so C_host is valid on return.
 * scratch_dev must hold awe_workspace_bytes + awe_host_staging_bytes bytes (256-B aligned).
 * For M >= 2048 the product is processed in blocks (row chunks of A; from N >= 4096 also column blocks
 * of B, uploaded alternately so that about as many rows of A as columns of B are on the device, each
 * arrival followed by one launch for the rectangle of C it completes and one copy back) so that the
 * copies to the device, the kernels and the copies back overlap; the copies run on two streams owned by
 * the handle (created on the first call) that are ordered after and before `stream` with events.
 * Pinned host memory is needed for that overlap; pageable memory works but serialises. */
awe_status_t awe_gemm_exact_host(awe_handle_t h, const void* A_host, awe_in_dtype_t a_dt, const void* B_host,
                                 awe_in_dtype_t b_dt, int64_t M, int64_t N, int64_t K, int enc, int modulus,
                                 void* C_host, awe_out_dtype_t out_dt, void* scratch_dev, size_t scratch_bytes,
                                 void* stream);

/* ---- Wide integers through a residue number system (Section 5.3; Table I, "FP64 significand").
 * The inputs are split into symmetric residues modulo pairwise coprime moduli, each residue product
 * runs as a mod-m product on the FP4 kernels, and the Chinese remainder theorem rebuilds the exact
 * integers.  The built-in set has 22 moduli (60 FP4 GEMMs) with product 2^122.86, which gives a
 * unique result whenever 2 K (2^(in_bits-1) - 1)^2 stays below it: in_bits = 54 up to K = 59,000.
 * Narrower inputs use a cheaper subset (awe_wide_select). */

/* The moduli of the built-in set: writes up to `capacity` of them to out (may be NULL), returns
 * how many there are.  Host only. */
int awe_wide_moduli(int32_t* out, int capacity);

/* The subset of the built-in moduli awe_gemm_exact_wide uses for inputs of `in_bits` bits and
 * reduction length K: the one with the fewest FP4 products whose product exceeds
 * 2 K (2^(in_bits-1) - 1)^2 (the selection problem of Section 5.3, solved exactly over the built-in
 * set).  Writes up to `capacity` moduli to out (may be NULL) and returns their number, 0 if even the
 * whole set is too small.  Host only. */
int awe_wide_select(int in_bits, int64_t K, int32_t* out, int capacity);

/* Bytes of scratch awe_gemm_exact_wide needs: residues of A and B (int8, one copy per modulus),
 * the residue products (int16 per modulus) and the plane workspace of one modulus. */
size_t awe_wide_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Symmetric residues of `count` 64-bit integers (|x| < 2^56) for every modulus of the set:
 * res_dev[t * count + i] = X_dev[i] mod m_t in [-floor(m_t/2), ceil(m_t/2) - 1], int8.  Elementwise, so
 * the residue arrays keep the layout of X.  X_dev 16-B aligned, res_dev 4-B aligned. */
awe_status_t awe_wide_residues(awe_handle_t h, const int64_t* X_dev, int64_t count, int8_t* res_dev, void* stream);

/* Chinese-remainder reconstruction: res_dev[t * count + i] (int16) is a residue of the unknown integer
 * x_i modulo m_t (the products deliver the symmetric one; any representative that fits 16 bits is
 * accepted); writes x_i, the representative with |x_i| <= prod(m)/2, as a
 * 128-bit two's-complement integer: out_dev[2 i] = low 64 bits, out_dev[2 i + 1] = high 64 bits. */
awe_status_t awe_wide_crt(awe_handle_t h, const int16_t* res_dev, int64_t count, int64_t* out_dev, void* stream);

/* C = A.B exactly for integer matrices whose entries satisfy |x| <= 2^(in_bits-1) - 1, in_bits <= 54.
 * A_dev: M x K int64 row-major, B_dev: K x N int64 row-major, C_dev: M x N 128-bit integers (two
 * int64 each, low word first).  AWE_ERR_RANGE if the moduli cannot hold the result for this K.
 * workspace_dev: awe_wide_workspace_bytes bytes, 256-B aligned.  Inputs outside the stated width
 * give an unspecified result (they are not checked on the device). */
awe_status_t awe_gemm_exact_wide(awe_handle_t h, const int64_t* A_dev, const int64_t* B_dev, int64_t M, int64_t N,
                                 int64_t K, int in_bits, int64_t* C_dev, void* workspace_dev, size_t workspace_bytes,
                                 void* stream);

/* Largest awe_workspace_bytes() a problem may need to go through awe_gemm_exact_static: 24 MiB,
 * e.g. INT8xINT8 with the 6-product encoding up to M = N = K = 2048. */
#define AWE_STATIC_WORKSPACE_BYTES (24u << 20)

/* The same product as awe_gemm_exact for callers that must not allocate device memory and so
 * cannot own a handle (awe_create calls cudaMalloc) or a workspace: code running inside a
 * runtime's execute hook that forbids allocation, in a process whose memory pool already holds
 * all of the GPU's memory so that cudaMalloc would fail, or on a latency-critical path that cannot
 * take cudaMalloc's device-wide synchronisation.  (The paper has no counterpart; it is a
 * deployment convenience.)  All device scratch -- planes, encode tables, status word -- comes from
 * one array built into the library image: AWE_STATIC_WORKSPACE_BYTES + ~200 KB, resident on every
 * GPU that loads the library until the process exits.  The call uses the CURRENT device, makes no
 * cudaMalloc / cudaFree, and enqueues the same kernels as awe_gemm_exact on `stream`.
 *   - A_dev, B_dev, C_dev, dtypes, sizes, enc, modulus, out_dt: exactly as for awe_gemm_exact
 *     (A: M x K, B: K x N, C: M x N, all row-major and dense).
 *   - AWE_ERR_WORKSPACE if awe_workspace_bytes(enc, modulus, M, N, K) exceeds
 *     AWE_STATIC_WORKSPACE_BYTES; nothing is enqueued then.  Encodings with 16-bit inputs are not
 *     served (AWE_ERR_UNSUPPORTED): their 32 KB tables have no room in the built-in array.
 *   - The first call on a device looks up the array's device address and the device's properties,
 *     clears the status word and (once per process) page-locks a small host mirror of the status words
 *     in place; the first use of an encoding on a device uploads its tables and waits for that copy
 *     (room for 96 tables per device).  These first calls synchronise `stream`, which a stream that is
 *     being captured does not allow.
 *   - Every call on a device shares the one array, which keeps the previous call's planes: calls
 *     whose kernels could overlap on the GPU (different streams, or several host threads) race
 *     and must be serialised by the caller.  Nothing in it needs to start at zero except the status
 *     word, which the library clears itself.
 *   - No call waits for the GPU.  Each call ends by enqueuing, on `stream`, a copy of the status word
 *     into the host mirror; a bounded device-side wait that expired during an earlier call is
 *     returned (as AWE_ERR_TIMEOUT, once) by the first later call that finds it there, and that call
 *     enqueues nothing but the clearing of the word: repeat it to get the product.  While `stream` is
 *     being captured the status word is neither copied nor looked at. */
awe_status_t awe_gemm_exact_static(const void* A_dev, awe_in_dtype_t a_dt, const void* B_dev, awe_in_dtype_t b_dt,
                                   int64_t M, int64_t N, int64_t K, int enc, int modulus, void* C_dev,
                                   awe_out_dtype_t out_dt, void* stream);

/* One raw FP4 product P = X.Y^T with FP32 accumulation over all of K in a single segment
 * (Algorithm 1's "FP4-GEMM" alone; Section 3.4 is the claim this lets a test probe).
 * planeX_dev: M x pitch bytes, planeY_dev: N x pitch bytes, pitch = round_up(K,256)/2, packed E2M1;
 * P_dev: M x N float, leading dimension ldp.  The values returned are in the doubled-integer
 * convention of Section 3.1 (each operand counted as an element of S). */
awe_status_t awe_fp4_product_raw(awe_handle_t h, const void* planeX_dev, const void* planeY_dev, int64_t M,
                                 int64_t N, int64_t K, float* P_dev, int64_t ldp, void* stream);

/* One raw FP8 (E4M3) product P = X.Y^T with FP32 accumulation over all of K in a single segment:
 * the FP8 products of the mixed 2 x FP8 + 1 x FP4 construction (Appendix A) alone, so that a test
 * can probe the exact-accumulation claim of Section 3.4 for this operand format too.
 * planeX_dev: M x pitch8 bytes, planeY_dev: N x pitch8 bytes, pitch8 = round_up(K,256), one E4M3
 * byte per element, zero-padded; both 256-byte aligned.  P_dev: M x N float, leading dimension
 * ldp; values are the plain products (E4M3 holds the integers themselves, no doubling). */
awe_status_t awe_fp8_product_raw(awe_handle_t h, const void* planeX_dev, const void* planeY_dev, int64_t M,
                                 int64_t N, int64_t K, float* P_dev, int64_t ldp, void* stream);

/* Stand-alone reconstruction (Algorithm 1, last step; Section 5.3 for the residue form) from the r
 * raw FP32 products of an encoding, e.g. written by awe_fp4_product_raw: product k is the M x N
 * matrix at P_dev + k * plane_stride with leading dimension ldp (floats, doubled-integer
 * convention).  Writes C = (sum_k l_k P_k) >> log2 D, or that sum mod m in the symmetric range, to
 * C_dev (leading dimension ldc, type out_dt).  The unfused counterpart of the epilogue of
 * awe_gemm_planes; every P_k must come from a single exact accumulation segment (K <= K*), and
 * AWE_C_I32 is subject to the same bound as there (D max|a| max|b| K < 2^31; not checked here, since
 * K is not an argument).  16-byte aligned P_dev and C rows with ldp, ldc, plane_stride multiples of 4
 * take the vector path. */
awe_status_t awe_reconstruct(awe_handle_t h, int enc, int modulus, const float* P_dev, int64_t plane_stride,
                             int64_t ldp, int64_t M, int64_t N, void* C_dev, awe_out_dtype_t out_dt, int64_t ldc,
                             void* stream);

/* Wait for `stream` and read the handle's device status word: AWE_OK, or AWE_ERR_TIMEOUT with
 * *site (may be NULL) naming the wait that gave up.  The word is cleared by the read. */
awe_status_t awe_last_device_status(awe_handle_t h, void* stream, int* site);

/* Self-test of the failure path: launches one warp that waits, with a budget of limit_us
 * microseconds (1 .. 1,000,000), on a barrier nothing signals.  The wait gives up, records
 * AWE_ERR_TIMEOUT with site 1000 in the status word and the kernel returns normally; the next
 * awe_last_device_status reports it and the handle stays usable.  Nothing faults or traps.
 * (No counterpart in the paper.) */
awe_status_t awe_selftest_bounded_wait(awe_handle_t h, int64_t limit_us, void* stream);

/* Diagnostic: the SM clock (MHz) at which the most recent GEMM launch on this handle actually ran,
 * measured inside the kernel by CTA 0 as elapsed SM cycles over elapsed nanoseconds.  Waits for
 * `stream`.  Lets a benchmark state the tensor-pipe peak at the delivered clock (the part is
 * power-capped under FP4 load).  (No counterpart in the paper.) */
awe_status_t awe_last_gemm_clock_mhz(awe_handle_t h, void* stream, double* mhz);

/* Number of this library's kernels launched through the handle since it was created. */
int64_t awe_launch_count(awe_handle_t h);

const char* awe_status_string(awe_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* AWE_H_ */

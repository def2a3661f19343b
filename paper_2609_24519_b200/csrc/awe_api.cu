// Handle management and the whole-procedure entry points (Algorithm 1 end to end).
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <initializer_list>
#include <new>

#include "awe_internal.h"

using namespace awe;

extern "C" awe_status_t awe_create(awe_handle_t* out, int device) {
    if (!out) return AWE_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return AWE_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return AWE_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return AWE_ERR_CUDA;
    if (prop.major != 10) return AWE_ERR_CUDA;  // the kernels are built for sm_100a only
    awe_ctx* h = new (std::nothrow) awe_ctx();
    if (!h) return AWE_ERR_CUDA;
    h->device = device;
    h->sm_count = prop.multiProcessorCount;
    h->lut_slots = kLutSlots;
    if (cudaMalloc(&h->status_dev, kStatusWords * sizeof(unsigned int)) != cudaSuccess ||
        cudaMemset(h->status_dev, 0, kStatusWords * sizeof(unsigned int)) != cudaSuccess ||
        cudaMalloc(&h->lut_arena_dev, (size_t)kLutSlots * 256 * sizeof(uint64_t)) != cudaSuccess ||
        cudaMalloc(&h->lut16_arena_dev, (size_t)kLut16Slots * 4096 * sizeof(uint64_t)) != cudaSuccess) {
        awe_destroy(h);
        return AWE_ERR_CUDA;
    }
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &h->encode_tiled, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !h->encode_tiled) {
        awe_destroy(h);
        return AWE_ERR_CUDA;
    }
    *out = h;
    return AWE_OK;
}

extern "C" awe_status_t awe_destroy(awe_handle_t h) {
    if (!h) return AWE_ERR_INVALID_ARG;
    cudaSetDevice(h->device);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    for (cudaEvent_t e : {h->ev_start, h->ev_b, h->ev_done})
        if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ev_a)
        if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ev_bcol)
        if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ev_c)
        if (e) cudaEventDestroy(e);
    if (h->status_dev) cudaFree(h->status_dev);
    if (h->lut_arena_dev) cudaFree(h->lut_arena_dev);
    if (h->lut16_arena_dev) cudaFree(h->lut16_arena_dev);
    delete h;
    return AWE_OK;
}

namespace awe {
awe_status_t device_lut(awe_ctx* h, int enc, int modulus, awe_side_t side, awe_in_dtype_t dt, cudaStream_t stream,
                        const uint64_t** out) {
    dt = table_dtype(dt);
    if (is_16bit(dt)) {  // 4096-entry tables live in their own arena (absent in the allocation-free context)
        if (!h->lut16_arena_dev) return AWE_ERR_UNSUPPORTED;
        for (size_t i = 0; i < h->slots16.size(); ++i)
            if (h->slots16[i].enc == enc && h->slots16[i].side == (int)side) {
                *out = h->lut16_arena_dev + i * 4096;
                return AWE_OK;
            }
        if ((int)h->slots16.size() >= kLut16Slots) return AWE_ERR_UNSUPPORTED;
        const SideTable* t16;
        if (!get_side_table(enc, modulus, side, dt, &t16)) return AWE_ERR_UNSUPPORTED;
        uint64_t* dst16 = h->lut16_arena_dev + h->slots16.size() * 4096;
        if (cudaMemcpyAsync(dst16, t16->lut.data(), 4096 * sizeof(uint64_t), cudaMemcpyHostToDevice, stream) !=
                cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
            return AWE_ERR_CUDA;
        h->slots16.push_back({enc, (int)side});
        *out = dst16;
        return AWE_OK;
    }
    for (size_t i = 0; i < h->slots.size(); ++i) {
        const auto& s = h->slots[i];
        if (s.enc == enc && s.modulus == modulus && s.side == (int)side && s.dt == (int)dt) {
            *out = h->lut_arena_dev + i * 256;
            return AWE_OK;
        }
    }
    if ((int)h->slots.size() >= h->lut_slots) return AWE_ERR_UNSUPPORTED;
    const SideTable* t;
    if (!get_side_table(enc, modulus, side, dt, &t)) return AWE_ERR_UNSUPPORTED;
    uint64_t* dst = h->lut_arena_dev + h->slots.size() * 256;
    // The table lives in host memory owned by the library for the life of the process, so the
    // copy may complete after this call returns.
    if (cudaMemcpyAsync(dst, t->lut.data(), 256 * sizeof(uint64_t), cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return AWE_ERR_CUDA;
    // Later calls may use another stream: make the table visible to all of them now.
    if (cudaStreamSynchronize(stream) != cudaSuccess) return AWE_ERR_CUDA;
    h->slots.push_back({enc, modulus, (int)side, (int)dt});
    *out = dst;
    return AWE_OK;
}
}  // namespace awe

static size_t out_elem_bytes(awe_out_dtype_t t) { return t == AWE_C_I64 ? 8 : (t == AWE_C_RES_I16 ? 2 : 4); }

extern "C" size_t awe_host_staging_bytes(int enc, int modulus, int64_t M, int64_t N, int64_t K,
                                         awe_out_dtype_t out_dt) {
    if (!awe_workspace_bytes(enc, modulus, M, N, K)) return 0;
    const awe_in_dtype_t na = natural_dtype(enc, AWE_SIDE_A), nb = natural_dtype(enc, AWE_SIDE_B);
    return (size_t)round_up(in_bytes(na, M * K), 256) + (size_t)round_up(in_bytes(nb, K * N), 256) +
           (size_t)round_up(M * N * (int64_t)out_elem_bytes(out_dt), 256);
}

extern "C" awe_status_t awe_gemm_exact(awe_handle_t h, const void* A_dev, awe_in_dtype_t a_dt, const void* B_dev,
                                       awe_in_dtype_t b_dt, int64_t M, int64_t N, int64_t K, int enc, int modulus,
                                       void* C_dev, awe_out_dtype_t out_dt, void* workspace_dev,
                                       size_t workspace_bytes, void* stream) {
    if (!h || !A_dev || !B_dev || !C_dev || !workspace_dev || M <= 0 || N <= 0 || K <= 0)
        return AWE_ERR_INVALID_ARG;
    const size_t need = awe_workspace_bytes(enc, modulus, M, N, K);
    if (!need) return AWE_ERR_UNSUPPORTED;
    if (workspace_bytes < need) return AWE_ERR_WORKSPACE;
    if ((uintptr_t)workspace_dev % 256) return AWE_ERR_ALIGNMENT;
    // Everything the later steps would reject is checked before the first launch.
    if ((int)out_dt < 0 || (int)out_dt > 3) return AWE_ERR_INVALID_ARG;
    awe_encoding_desc d;
    awe_status_t s = awe_encoding_info(enc, modulus, &d);
    if (s != AWE_OK) return s;
    if ((d.modulus != 0) != (out_dt == AWE_C_RES_I16 || out_dt == AWE_C_RES_I32)) return AWE_ERR_UNSUPPORTED;
    if ((uintptr_t)C_dev % out_elem_bytes(out_dt)) return AWE_ERR_ALIGNMENT;
    const SideTable* t;
    if (!get_side_table(enc, modulus, AWE_SIDE_A, a_dt, &t) || !get_side_table(enc, modulus, AWE_SIDE_B, b_dt, &t))
        return AWE_ERR_UNSUPPORTED;
    if (out_dt == AWE_C_I32 && !i32_output_fits(d, K)) return AWE_ERR_RANGE;
    // both tables are on the device (or the arena is known to be full) before the first launch
    const uint64_t* lut;
    if ((s = device_lut(h, enc, modulus, AWE_SIDE_A, a_dt, (cudaStream_t)stream, &lut)) != AWE_OK ||
        (s = device_lut(h, enc, modulus, AWE_SIDE_B, b_dt, (cudaStream_t)stream, &lut)) != AWE_OK)
        return s;

    uint8_t* pa = (uint8_t*)workspace_dev;
    uint8_t* pb = pa + round_up((int64_t)awe_planes_bytes(enc, modulus, AWE_SIDE_A, M, K), 256);
    if ((s = awe_encode(h, enc, modulus, AWE_SIDE_A, A_dev, a_dt, AWE_ROWMAJOR_RxK, M, K, K, pa, stream)) != AWE_OK)
        return s;
    if ((s = awe_encode(h, enc, modulus, AWE_SIDE_B, B_dev, b_dt, AWE_ROWMAJOR_KxR, N, K, N, pb, stream)) != AWE_OK)
        return s;
    return awe_gemm_planes(h, enc, modulus, pa, pb, M, N, K, C_dev, out_dt, N, 0, stream);
}

extern "C" awe_status_t awe_gemm_exact_host(awe_handle_t h, const void* A_host, awe_in_dtype_t a_dt,
                                            const void* B_host, awe_in_dtype_t b_dt, int64_t M, int64_t N, int64_t K,
                                            int enc, int modulus, void* C_host, awe_out_dtype_t out_dt,
                                            void* scratch_dev, size_t scratch_bytes, void* stream) {
    if (!h || !A_host || !B_host || !C_host || !scratch_dev || M <= 0 || N <= 0 || K <= 0)
        return AWE_ERR_INVALID_ARG;
    if ((int)out_dt < 0 || (int)out_dt > 3) return AWE_ERR_INVALID_ARG;
    const size_t ws = awe_workspace_bytes(enc, modulus, M, N, K);
    const size_t staging = awe_host_staging_bytes(enc, modulus, M, N, K, out_dt);
    if (!ws || !staging) return AWE_ERR_UNSUPPORTED;
    if (scratch_bytes < ws + staging) return AWE_ERR_WORKSPACE;
    if ((uintptr_t)scratch_dev % 256) return AWE_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* base = (uint8_t*)scratch_dev;
    // staging is sized for the natural container of the encoding; a packed 4-bit operand needs less
    if (in_elem_nibbles(a_dt) > in_elem_nibbles(natural_dtype(enc, AWE_SIDE_A)) ||
        in_elem_nibbles(b_dt) > in_elem_nibbles(natural_dtype(enc, AWE_SIDE_B)))
        return AWE_ERR_UNSUPPORTED;
    if ((a_dt == AWE_I4_PACKED && (K & 1)) || (b_dt == AWE_I4_PACKED && (N & 1))) return AWE_ERR_INVALID_ARG;
    uint8_t* dA = base + round_up((int64_t)ws, 256);
    uint8_t* dB = dA + round_up(in_bytes(natural_dtype(enc, AWE_SIDE_A), M * K), 256);
    uint8_t* dC = dB + round_up(in_bytes(natural_dtype(enc, AWE_SIDE_B), K * N), 256);
    const size_t elem = out_elem_bytes(out_dt);
    // Everything awe_gemm_exact would reject is rejected here, before any copy is enqueued.
    awe_encoding_desc d;
    awe_status_t s = awe_encoding_info(enc, modulus, &d);
    if (s != AWE_OK) return s;
    if ((d.modulus != 0) != (out_dt == AWE_C_RES_I16 || out_dt == AWE_C_RES_I32)) return AWE_ERR_UNSUPPORTED;
    const SideTable* tbl;
    if (!get_side_table(enc, modulus, AWE_SIDE_A, a_dt, &tbl) || !get_side_table(enc, modulus, AWE_SIDE_B, b_dt, &tbl))
        return AWE_ERR_UNSUPPORTED;
    if (out_dt == AWE_C_I32 && !i32_output_fits(d, K)) return AWE_ERR_RANGE;
    const uint64_t* lut;
    if ((s = device_lut(h, enc, modulus, AWE_SIDE_A, a_dt, st, &lut)) != AWE_OK ||
        (s = device_lut(h, enc, modulus, AWE_SIDE_B, b_dt, st, &lut)) != AWE_OK)
        return s;

    // The product is cut into blocks so that the copies to the device, the kernels and the copies back
    // overlap (the two copy directions run on their own streams).  The result is twice the bytes of the
    // operands, so the copy back is the long pole: it should start early and never wait.  With a rows
    // of A and b columns of B on the device, a x b entries of C can be computed, so the uploads alternate
    // between row chunks of A and column blocks of B to keep a and b about equal (column block 0 first,
    // small row chunks at the start so that the first block of C leaves after about 0.4 ms).  Each
    // arrival makes one new rectangle of C computable -- the new rows against all columns present, or
    // all rows present against the new columns: one launch on planes that every chunk is encoded into
    // in place, and one two-dimensional copy back.  Small problems go through in one piece.
    int64_t row_edge[awe_ctx::kMaxHostChunks + 1], col_edge[awe_ctx::kMaxHostColBlocks + 1];
    int n_row = 0, n_col = 0;
    auto cut = [](int64_t total, const int64_t* first, int n_first, int64_t rest, int max_parts, int64_t* edge) {
        int n = 0;
        int64_t at = 0;
        edge[0] = 0;
        while (at < total) {
            int64_t step = n < n_first ? first[n] : rest;
            // the last part takes what is left (also when the table of parts is used up)
            if (n + 1 == max_parts || total - at < step + step / 2) step = total - at;
            at += step;
            edge[++n] = at;
        }
        return n;
    };
    if (M >= 2048 && N >= 4096) {
        const int64_t rows_first[5] = {512, 512, 1024, 1024, 1024}, cols_first[3] = {2048, 1024, 1024};
        n_row = cut(M, rows_first, 5, 2048, awe_ctx::kMaxHostChunks, row_edge);
        n_col = cut(N, cols_first, 3, 2048, awe_ctx::kMaxHostColBlocks, col_edge);
    } else {
        // few rows or columns: row chunks of at least 1024 still overlap the copies, no column blocks
        const int chunks = (int)std::max<int64_t>(1, std::min<int64_t>(awe_ctx::kMaxHostChunks, M / 1024));
        const int64_t per = chunks == 1 ? M : round_up((M + chunks - 1) / chunks, 256);
        n_row = cut(M, nullptr, 0, per, awe_ctx::kMaxHostChunks, row_edge);
        n_col = 1;
        col_edge[0] = 0;
        col_edge[1] = N;
    }
    if (!h->copy_in) {
        bool ok = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&h->ev_b, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&h->ev_done, cudaEventDisableTiming) == cudaSuccess;
        for (cudaEvent_t& e : h->ev_a) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
        for (cudaEvent_t& e : h->ev_bcol) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
        for (cudaEvent_t& e : h->ev_c) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return AWE_ERR_CUDA;
    }
#define AWE_CU(x) do { if ((x) != cudaSuccess) return AWE_ERR_CUDA; } while (0)
    uint8_t* pa = base;
    uint8_t* pb = base + round_up((int64_t)awe_planes_bytes(enc, modulus, AWE_SIDE_A, M, K), 256);
    const int64_t nib_b = in_elem_nibbles(b_dt);  // half-bytes per element of B
    AWE_CU(cudaEventRecord(h->ev_start, st));
    AWE_CU(cudaStreamWaitEvent(h->copy_in, h->ev_start, 0));
    AWE_CU(cudaStreamWaitEvent(h->copy_out, h->ev_start, 0));
    // Order of arrival: column block 0, then whichever operand has fewer rows (columns) on the device.
    struct Arrival { bool is_a; int index; };
    Arrival order[awe_ctx::kMaxHostChunks + awe_ctx::kMaxHostColBlocks];
    int n_order = 0;
    {
        int i = 0, j = 0;
        order[n_order++] = {false, j++};
        while (i < n_row || j < n_col) {
            const bool take_a = i < n_row && (j >= n_col || row_edge[i] < col_edge[j]);
            order[n_order++] = take_a ? Arrival{true, i++} : Arrival{false, j++};
        }
    }
    for (int o = 0; o < n_order; ++o) {
        if (order[o].is_a) {
            const int64_t r0 = row_edge[order[o].index], rows = row_edge[order[o].index + 1] - r0;
            AWE_CU(cudaMemcpyAsync(dA + (size_t)in_bytes(a_dt, r0 * K), (const uint8_t*)A_host + (size_t)in_bytes(a_dt, r0 * K),
                                   (size_t)in_bytes(a_dt, rows * K), cudaMemcpyHostToDevice, h->copy_in));
            AWE_CU(cudaEventRecord(h->ev_a[order[o].index], h->copy_in));
        } else {
            const int64_t c0 = col_edge[order[o].index], cols = col_edge[order[o].index + 1] - c0;
            if (n_col == 1) {
                AWE_CU(cudaMemcpyAsync(dB, B_host, (size_t)in_bytes(b_dt, K * N), cudaMemcpyHostToDevice, h->copy_in));
            } else {
                AWE_CU(cudaMemcpy2DAsync(dB + c0 * nib_b / 2, (size_t)(N * nib_b / 2), (const uint8_t*)B_host + c0 * nib_b / 2,
                                         (size_t)(N * nib_b / 2), (size_t)(cols * nib_b / 2), (size_t)K,
                                         cudaMemcpyHostToDevice, h->copy_in));
            }
            AWE_CU(cudaEventRecord(h->ev_bcol[order[o].index], h->copy_in));
        }
    }
    // C rows [r0, r0 + rows) x columns [c0, c0 + cols): product on the planes present, then the copy back
    auto region = [&](int slot, int64_t r0, int64_t rows, int64_t c0, int64_t cols) -> awe_status_t {
        if (rows <= 0 || cols <= 0) return AWE_OK;
        uint8_t* c_dev = dC + ((size_t)r0 * N + c0) * elem;
        awe_status_t rs = gemm_planes_window(h, enc, modulus, PlaneWindow{pa, M, r0}, PlaneWindow{pb, N, c0}, rows, cols, K,
                                             c_dev, out_dt, N, 0, stream);
        if (rs != AWE_OK) return rs;
        AWE_CU(cudaEventRecord(h->ev_c[slot], st));
        AWE_CU(cudaStreamWaitEvent(h->copy_out, h->ev_c[slot], 0));
        uint8_t* c_host = (uint8_t*)C_host + ((size_t)r0 * N + c0) * elem;
        if (cols == N) {
            AWE_CU(cudaMemcpyAsync(c_host, c_dev, (size_t)rows * N * elem, cudaMemcpyDeviceToHost, h->copy_out));
        } else {
            AWE_CU(cudaMemcpy2DAsync(c_host, (size_t)N * elem, c_dev, (size_t)N * elem, (size_t)cols * elem, (size_t)rows,
                                     cudaMemcpyDeviceToHost, h->copy_out));
        }
        return AWE_OK;
    };
    int64_t a_done = 0, b_done = 0;
    for (int o = 0; o < n_order; ++o) {
        if (order[o].is_a) {
            const int64_t r0 = row_edge[order[o].index], rows = row_edge[order[o].index + 1] - r0;
            AWE_CU(cudaStreamWaitEvent(st, h->ev_a[order[o].index], 0));
            if ((s = encode_window(h, enc, modulus, AWE_SIDE_A, dA + (size_t)in_bytes(a_dt, r0 * K), a_dt, AWE_ROWMAJOR_RxK,
                                   rows, K, K, PlaneWindow{pa, M, r0}, stream)) != AWE_OK)
                return s;
            if ((s = region(o, r0, rows, 0, b_done)) != AWE_OK) return s;
            a_done = r0 + rows;
        } else {
            const int64_t c0 = col_edge[order[o].index], cols = col_edge[order[o].index + 1] - c0;
            AWE_CU(cudaStreamWaitEvent(st, h->ev_bcol[order[o].index], 0));
            if ((s = encode_window(h, enc, modulus, AWE_SIDE_B, dB + c0 * nib_b / 2, b_dt, AWE_ROWMAJOR_KxR, cols, K, N,
                                   PlaneWindow{pb, N, c0}, stream)) != AWE_OK)
                return s;
            if ((s = region(o, 0, a_done, c0, cols)) != AWE_OK) return s;
            b_done = c0 + cols;
        }
    }
    AWE_CU(cudaEventRecord(h->ev_done, h->copy_out));
    AWE_CU(cudaStreamWaitEvent(st, h->ev_done, 0));
    AWE_CU(cudaStreamSynchronize(st));
#undef AWE_CU
    return AWE_OK;
}

extern "C" awe_status_t awe_last_device_status(awe_handle_t h, void* stream, int* site) {
    if (!h) return AWE_ERR_INVALID_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return AWE_ERR_CUDA;
    unsigned int w[2] = {0, 0};
    if (cudaMemcpy(w, h->status_dev, sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess) return AWE_ERR_CUDA;
    if (w[0] != 0 && cudaMemset(h->status_dev, 0, sizeof(w)) != cudaSuccess) return AWE_ERR_CUDA;
    if (site) *site = (int)w[1];
    return (awe_status_t)w[0];
}

extern "C" awe_status_t awe_last_gemm_clock_mhz(awe_handle_t h, void* stream, double* mhz) {
    if (!h || !mhz) return AWE_ERR_INVALID_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return AWE_ERR_CUDA;
    unsigned long long w[2] = {0, 0};
    if (cudaMemcpy(w, h->status_dev + 2, sizeof(w), cudaMemcpyDeviceToHost) != cudaSuccess) return AWE_ERR_CUDA;
    *mhz = w[1] ? (double)w[0] / (double)w[1] * 1e3 : 0.0;
    return AWE_OK;
}

extern "C" int64_t awe_launch_count(awe_handle_t h) { return h ? h->launches : -1; }

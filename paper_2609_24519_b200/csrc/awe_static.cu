// awe_gemm_exact_static: the whole exact product for callers that may not allocate device memory.
//
// Every byte of device scratch this entry point needs -- the packed planes of both operands,
// the encode tables and the status word -- lives in one file-scope __device__ array that is part
// of the library image, so the call makes no cudaMalloc / cudaFree and needs no handle (a handle
// owns cudaMalloc'd memory).  The kernels are the ones awe_gemm_exact launches; only the source of
// their scratch pointers differs.
//
// In host code the array's name is only a host-side stand-in for the symbol: its device address
// is obtained once per device with cudaGetSymbolAddress, while that device is current, and that
// address is what the kernels receive.
#include <cstring>

#include "awe_internal.h"

using namespace awe;

namespace {

constexpr size_t kTableBytes = (size_t)kStaticLutSlots * 256 * sizeof(uint64_t);
constexpr size_t kStatusBytes = 256;
constexpr size_t kScratchBytes = (size_t)AWE_STATIC_WORKSPACE_BYTES + kTableBytes + kStatusBytes;

// Layout: [planes of A, planes of B | encode tables | status word].  Held by every GPU that loads
// the library, from load until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;

struct DeviceState {
    bool ready = false;
    unsigned char* base = nullptr;  // device address of g_static_scratch on this device
    awe_ctx ctx;                    // host-side bookkeeping only; owns no device allocation
};

DeviceState g_state[kMaxDevices];
std::mutex g_setup_mu;

// Host mirror of each device's status word.  Every call ends with an asynchronous copy of the word
// into its device's slot, on the caller's stream, and the next call only looks at the slot: no call
// ever waits for the GPU to learn about an earlier one.  The slots are ordinary library memory,
// page-locked in place at the first set-up (nothing is allocated) so that those copies really are
// asynchronous; if the lock is refused the mirror is not used and expired waits go unreported.
struct alignas(64) StatusSlot {
    volatile unsigned int word[2];  // status, site
    unsigned int pad[14];
};
alignas(4096) StatusSlot g_status_mirror[kMaxDevices];
bool g_mirror_tried = false, g_mirror_locked = false;

// One-time set-up for the current device.  Not allocating, but it does query the device and
// resolves the symbol, so it belongs before any stream capture.
awe_status_t setup_device(int device, cudaStream_t stream, DeviceState** out) {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    DeviceState& s = g_state[device];
    if (!s.ready) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
            return AWE_ERR_CUDA;
        if (major != 10) return AWE_ERR_CUDA;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return AWE_ERR_CUDA;
        s.base = (unsigned char*)ptr;
        s.ctx.device = device;
        s.ctx.sm_count = sms;
        s.ctx.lut_arena_dev = (uint64_t*)(s.base + AWE_STATIC_WORKSPACE_BYTES);
        s.ctx.lut_slots = kStaticLutSlots;
        s.ctx.status_dev = (unsigned int*)(s.base + AWE_STATIC_WORKSPACE_BYTES + kTableBytes);
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &s.ctx.encode_tiled, cudaEnableDefault, &q) !=
                cudaSuccess ||
            q != cudaDriverEntryPointSuccess || !s.ctx.encode_tiled)
            return AWE_ERR_CUDA;
        if (!g_mirror_tried) {
            g_mirror_tried = true;
            g_mirror_locked =
                cudaHostRegister(g_status_mirror, sizeof(g_status_mirror), cudaHostRegisterPortable) == cudaSuccess;
            if (!g_mirror_locked) cudaGetLastError();  // the refusal is not this call's error
        }
        // The array keeps whatever an earlier process image or call left: the status word must start at zero.
        if (cudaMemsetAsync(s.ctx.status_dev, 0, kStatusBytes, stream) != cudaSuccess) return AWE_ERR_CUDA;
        s.ready = true;
    }
    *out = &s;
    return AWE_OK;
}

}  // namespace

extern "C" awe_status_t awe_gemm_exact_static(const void* A_dev, awe_in_dtype_t a_dt, const void* B_dev,
                                              awe_in_dtype_t b_dt, int64_t M, int64_t N, int64_t K, int enc,
                                              int modulus, void* C_dev, awe_out_dtype_t out_dt, void* stream) {
    if (!A_dev || !B_dev || !C_dev || M <= 0 || N <= 0 || K <= 0) return AWE_ERR_INVALID_ARG;
    const size_t need = awe_workspace_bytes(enc, modulus, M, N, K);
    if (!need) return AWE_ERR_UNSUPPORTED;
    if (need > (size_t)AWE_STATIC_WORKSPACE_BYTES) return AWE_ERR_WORKSPACE;  // beyond the built-in scratch
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return AWE_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    DeviceState* s = nullptr;
    awe_status_t rc = setup_device(device, st, &s);
    if (rc != AWE_OK) return rc;
    // While `stream` is being captured nothing may be read back or compared on the host: the status
    // word is left alone and only the kernels are recorded.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) return AWE_ERR_CUDA;
    const bool report = g_mirror_locked && cap == cudaStreamCaptureStatusNone;
    // A wait that gave up inside an earlier call's kernels shows up in the host mirror once that
    // call's trailing copy has run; the call that sees it clears the word, returns the status and does
    // no other work.
    if (report) {
        StatusSlot& slot = g_status_mirror[device];
        const unsigned int seen = slot.word[0];
        if (seen != 0) {
            slot.word[0] = 0;
            slot.word[1] = 0;
            if (cudaMemsetAsync(s->ctx.status_dev, 0, 2 * sizeof(unsigned int), st) != cudaSuccess) return AWE_ERR_CUDA;
            return (awe_status_t)seen;
        }
    }
    // Planes are rewritten in full (padding included) by the encode kernels, so nothing else in the
    // array needs clearing between calls.
    rc = awe_gemm_exact(&s->ctx, A_dev, a_dt, B_dev, b_dt, M, N, K, enc, modulus, C_dev, out_dt, s->base,
                        (size_t)AWE_STATIC_WORKSPACE_BYTES, stream);
    if (rc == AWE_OK && report &&
        cudaMemcpyAsync((void*)g_status_mirror[device].word, s->ctx.status_dev, 2 * sizeof(unsigned int),
                        cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return AWE_ERR_CUDA;
    return rc;
}

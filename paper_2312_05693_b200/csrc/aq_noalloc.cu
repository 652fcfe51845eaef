// aq_linear_w4a8_noalloc: the W4A8 layer for callers that may not allocate device memory
// (programs inside a memory pool that already owns the whole device, hosts that forbid
// cudaMalloc after start-up, real-time loops). The scratch the layer needs, normally a
// workspace passed by the caller, is a fixed device array compiled into the library.
#include "aq_common.cuh"

namespace {

// The layer's scratch: control block + int8 activation codes (+ small per-row scratch), laid
// out exactly as aq_linear_w4a8 lays out a caller's workspace. Held by every GPU that loads
// the library until the process exits; shared by all calls on that GPU.
static __device__ __align__(256) unsigned char g_noalloc_scratch[AQ_NOALLOC_SCRATCH_BYTES];

// Device address of the array on each device, looked up once per device. In host code the
// name g_noalloc_scratch is only a stand-in for the symbol, never a pointer a kernel may use.
// Atomic: two host threads may make their first call on a device at the same time (both then
// look the address up and store the same value).
std::atomic<void*> g_scratch_addr[aq::kMaxDevices];

// The handle's device must be current; returns the array's address there (looked up on first use).
int scratch_address(aq_handle_t h, void** out) {
    const int dev = aq::handle_device(h);
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) { aq::handle_record_cuda_error(h, e); return AQ_ERR_CUDA; }
    if (dev < 0 || dev >= aq::kMaxDevices || cur != dev) return AQ_ERR_INVALID_ARG;
    void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!p) {
        // one-time set-up on this device (it is current): ask the runtime where the array lives
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) { aq::handle_record_cuda_error(h, e); return AQ_ERR_CUDA; }
        g_scratch_addr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return AQ_OK;
}

}  // namespace

extern "C" int aq_linear_w4a8_noalloc(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                                      const void* w_scales, int N, int group_size, int scale_mode,
                                      int clip_shift_or_exp, void* y_fp16, void* stream) {
    if (!h) return AQ_ERR_INVALID_ARG;
    // Only the part of the workspace the layer cannot do without counts against the array: control
    // block, codes, per-row scratch, per-channel offsets. The optional area for partial sums of shared
    // tiles (per-group scales) is whatever is left; with less than the kernel would like it simply
    // shares no tile.
    const size_t need = aq_workspace_min_bytes(M, K, N, group_size);
    if (need == 0) return AQ_ERR_SHAPE;
    if (need > AQ_NOALLOC_SCRATCH_BYTES) return AQ_ERR_TOO_LARGE;
    void* scratch = nullptr;
    const int rc = scratch_address(h, &scratch);
    if (rc != AQ_OK) return rc;
    // aq_linear_w4a8 clears the control block (the only part that must start at zero) itself;
    // the codes are fully rewritten before they are read.
    return aq_linear_w4a8(h, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp,
                          nullptr, y_fp16, nullptr, scratch, AQ_NOALLOC_SCRATCH_BYTES, stream);
}

extern "C" int aq_check_noalloc(aq_handle_t h, void* stream) {
    if (!h) return AQ_ERR_INVALID_ARG;
    void* scratch = nullptr;
    const int rc = scratch_address(h, &scratch);
    if (rc != AQ_OK) return rc;
    return aq_check_workspace(h, scratch, stream);
}

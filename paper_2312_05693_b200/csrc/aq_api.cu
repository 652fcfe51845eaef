// C ABI of the library: argument checks, workspace carving and kernel sequencing. Every
// step of the layer runs in the kernels of the sibling files; nothing here computes.
#include <new>

#include <math.h>

#include "aq_common.cuh"

struct aq_context {
    aq::DeviceInfo dev;
    int last_cuda_error;
    int kernel_choice;
    int weights_stable;
};

namespace {

using namespace aq;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }

int cuda_fail(aq_handle_t h, cudaError_t e) {
    if (h) h->last_cuda_error = (int)e;
    return AQ_ERR_CUDA;
}

int check_shape(int M, int K, int N, int group) {
    if (M < 1 || N < 1) return AQ_ERR_SHAPE;
    if (K < 32 || K > 65536 || K % 32 != 0) return AQ_ERR_SHAPE;
    if (group != 0 && group != 128) return AQ_ERR_SHAPE;
    if (group == 128 && K % 128 != 0) return AQ_ERR_SHAPE;
    if ((size_t)M * (size_t)N > ((size_t)1 << 40)) return AQ_ERR_SHAPE;
    return AQ_OK;
}

struct Workspace {
    Control* ctl;
    int8_t* codes;
    void* scratch;
    size_t scratch_bytes;
    float* chan_offset;
    float* split_scratch;
    size_t split_bytes;
};

// [control block][codes M*K][kernel scratch, M bytes][per-channel offsets of the zero-point variant, N floats]
// [fp32 partial outputs of tiles that two CTAs share in the tensor kernel, sized for a 148-SM B200; a
// device that would need more simply shares no tile]
constexpr int kPlannedSmCount = 148;
// what every call needs
size_t workspace_min_bytes(int M, int K, int N) {
    return sizeof(Control) + up256((size_t)M * K) + up256((size_t)M) + up256((size_t)N * sizeof(float));
}
// plus the optional area that lets the per-group tensor kernel share the tiles of a partial last round
size_t workspace_bytes(int M, int K, int N, int group) {
    return workspace_min_bytes(M, K, N) + up256(tensor_split_scratch_bytes(M, K, N, group, kPlannedSmCount));
}

Workspace carve(void* ws, int M, int K, int N, size_t total_bytes) {
    Workspace w;
    uint8_t* b = static_cast<uint8_t*>(ws);
    w.ctl = reinterpret_cast<Control*>(b);
    w.codes = reinterpret_cast<int8_t*>(b + sizeof(Control));
    w.scratch = b + sizeof(Control) + up256((size_t)M * K);
    w.scratch_bytes = up256((size_t)M);
    w.chan_offset = reinterpret_cast<float*>(b + sizeof(Control) + up256((size_t)M * K) + up256((size_t)M));
    const size_t used = workspace_min_bytes(M, K, N);
    w.split_scratch = reinterpret_cast<float*>(b + used);
    w.split_bytes = total_bytes > used ? total_bytes - used : 0;
    return w;
}

int kernel_for(aq_handle_t h, int M) {
    const int choice = h->kernel_choice;
    return choice == AQ_KERNEL_AUTO ? (M <= 16 ? AQ_KERNEL_DECODE : AQ_KERNEL_TENSOR) : choice;
}

int run_gemm(aq_handle_t h, const GemmArgs& g, cudaStream_t stream) {
    const int choice = kernel_for(h, g.M);
    GemmArgs a = g;
    a.weights_stable = h->weights_stable != 0;
    const cudaError_t e = choice == AQ_KERNEL_DECODE ? launch_gemm_decode(a, h->dev, stream)
                                                     : launch_gemm_tensor(a, h->dev, stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

// Scale + codes with the kernel that fits the size and the scale mode. `alpha` / `k_max`: TRIP factors
// or NULL / 0.
cudaError_t quantize_dispatch(aq_handle_t h, const __half* xh, int M, int K, const int32_t* row_idx, int bits,
                              int scale_mode, int clip_shift_or_exp, Control* ctl, int8_t* q, int32_t* scale_exp_out,
                              const uint8_t* alpha, int k_max, cudaStream_t stream) {
    if (quantize_small_fits(M, K))
        // small activations (decode): one kernel finds the scale, writes the codes and initialises
        // the control block
        return launch_quantize_small(xh, M, K, row_idx, bits, scale_mode, clip_shift_or_exp, ctl, q, scale_exp_out,
                                     stream, alpha, k_max, h->weights_stable != 0);
    const cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e != cudaSuccess) return e;
    if (scale_mode == AQ_SCALE_DYNAMIC)
        return launch_quantize_fused(xh, M, K, row_idx, bits, clip_shift_or_exp, ctl, q, scale_exp_out, h->dev, stream,
                                     alpha, k_max);
    return launch_quantize(xh, M, K, row_idx, bits, scale_mode, clip_shift_or_exp, ctl, q, scale_exp_out, h->dev,
                           stream, alpha, k_max);
}

bool trip_args_ok(const uint8_t* alpha, int k_max) { return alpha && k_max >= 0 && k_max <= 4; }

int linear_impl(aq_handle_t h, int bits, const void* x, int M, int K, const void* w_packed,
                const void* w_scales, int N, int group, int scale_mode, int clip_shift_or_exp,
                const int32_t* row_idx, void* y, int32_t* acc_dump, void* workspace, size_t workspace_bytes_,
                void* stream_, const uint8_t* alpha = nullptr, int k_max = 0, const float* w_offsets = nullptr,
                int8_t* q_next = nullptr, int next_bits = 8, int next_exp = 0, bool next_packed = false) {
    if (!h || !x || !w_packed || !w_scales || (!y && !q_next)) return AQ_ERR_INVALID_ARG;
    if (next_packed && (!q_next || next_bits != 4)) return AQ_ERR_INVALID_ARG;
    if (next_packed && N % 32 != 0) return AQ_ERR_SHAPE;
    if (next_packed && !aligned(q_next, 16)) return AQ_ERR_ALIGNMENT;
    if (q_next && ((next_bits != 8 && next_bits != 4) || next_exp < -40 || next_exp > 40 || w_offsets))
        return AQ_ERR_INVALID_ARG;
    if (scale_mode != AQ_SCALE_DYNAMIC && scale_mode != AQ_SCALE_STATIC) return AQ_ERR_INVALID_ARG;
    if (scale_mode == AQ_SCALE_DYNAMIC && (clip_shift_or_exp < 0 || clip_shift_or_exp > 16)) return AQ_ERR_INVALID_ARG;
    if (scale_mode == AQ_SCALE_STATIC && (clip_shift_or_exp < -40 || clip_shift_or_exp > 40)) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, N, group);
    if (s != AQ_OK) return s;
    if (!workspace || workspace_bytes_ < workspace_min_bytes(M, K, N)) return AQ_ERR_WORKSPACE;
    if (!aligned(x, 16) || !aligned(w_packed, 16) || !aligned(w_scales, 2) || (y && !aligned(y, 2)) ||
        !aligned(workspace, 256) || (acc_dump && !aligned(acc_dump, 4)) || (row_idx && !aligned(row_idx, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const Workspace w = carve(workspace, M, K, N, workspace_bytes_);
    const __half* xh = static_cast<const __half*>(x);
    if (alpha && !aligned(alpha, 16)) return AQ_ERR_ALIGNMENT;
    cudaError_t e = cudaSuccess;
    // a single row on the few-row kernel: that kernel finds the scale and makes the codes itself
    const bool fuse = !w_offsets && !alpha && kernel_for(h, M) == AQ_KERNEL_DECODE &&
                      decode_can_fuse_quantize(M, K, N, group, h->dev.sm_count);
    if (fuse) {
    } else if (w_offsets) {
        // zero-point variant: min / max, then e, zp and codes; then the per-channel term -(zp - 2^(b-1)) * r[n]
        if (!aligned(w_offsets, 4)) return AQ_ERR_ALIGNMENT;
        e = cudaMemsetAsync(w.ctl, 0, sizeof(Control), stream);
        if (e == cudaSuccess)
            e = launch_quantize_asym(xh, M, K, row_idx, bits, w.ctl, w.codes, nullptr, nullptr, h->dev, stream);
        if (e == cudaSuccess) e = launch_chan_offsets(w_offsets, N, bits, w.ctl, w.chan_offset, stream);
    } else {
        e = quantize_dispatch(h, xh, M, K, row_idx, bits, scale_mode, clip_shift_or_exp, w.ctl, w.codes, nullptr, alpha,
                              k_max, stream);
    }
    if (e != cudaSuccess) return cuda_fail(h, e);
    GemmArgs g;
    g.q = w.codes; g.M = M; g.K = K; g.N = N; g.group = group;
    g.w_packed = static_cast<const uint8_t*>(w_packed);
    g.w_scales = static_cast<const __half*>(w_scales);
    g.scale_exp = &w.ctl->scale_exp;
    g.y = static_cast<__half*>(y);
    g.acc_dump = acc_dump;
    g.ctl = w.ctl; g.scratch = w.scratch; g.scratch_bytes = w.scratch_bytes;
    g.split_scratch = w.split_scratch; g.split_bytes = w.split_bytes;
    g.chan_offset = w_offsets ? w.chan_offset : nullptr;
    g.q_next = q_next; g.next_bits = next_bits; g.next_exp = next_exp;
    g.next_packed = next_packed;
    g.after_quantize = !fuse;
    if (fuse) {
        g.fuse_x = xh; g.fuse_row_idx = row_idx; g.fuse_bits = bits; g.fuse_scale_mode = scale_mode;
        g.fuse_clip_shift_or_exp = clip_shift_or_exp;
    }
    return run_gemm(h, g, stream);
}

}  // namespace

extern "C" {

const char* aq_status_string(int status) {
    switch (status) {
        case AQ_OK: return "ok";
        case AQ_ERR_INVALID_ARG: return "invalid argument";
        case AQ_ERR_SHAPE: return "unsupported shape";
        case AQ_ERR_ALIGNMENT: return "misaligned pointer";
        case AQ_ERR_WORKSPACE: return "workspace missing or too small";
        case AQ_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.0";
        case AQ_ERR_CUDA: return "CUDA call failed";
        case AQ_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel gave up";
        case AQ_ERR_TOO_LARGE: return "sizes exceed the library's built-in scratch buffer";
        default: return "unknown status";
    }
}

int aq_version(void) { return 200; }

// 1: blocks of 128 channels x 128 k, 16-byte units of 32 codes, nibble planes (see aq_common.cuh).
// 2: the same, with K padded to a multiple of 128 by zero codes (identical to 1 when K % 128 == 0).
int aq_packed_w4_layout_version(void) { return 2; }

int aq_create(aq_handle_t* out, int device) {
    if (!out) return AQ_ERR_INVALID_ARG;
    *out = nullptr;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) return AQ_ERR_CUDA;
    if (prop.major != 10 || prop.minor != 0) return AQ_ERR_UNSUPPORTED_DEVICE;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) return AQ_ERR_CUDA;
    aq_context* c = new (std::nothrow) aq_context();
    if (!c) return AQ_ERR_INVALID_ARG;
    c->dev.device = device;
    c->dev.sm_count = prop.multiProcessorCount;
    c->dev.cc_major = prop.major;
    c->dev.cc_minor = prop.minor;
    c->dev.smem_optin = prop.sharedMemPerBlockOptin;
    c->dev.encode_tiled = fn;
    c->last_cuda_error = 0;
    c->kernel_choice = AQ_KERNEL_AUTO;
    c->weights_stable = 0;
    *out = c;
    return AQ_OK;
}

int aq_destroy(aq_handle_t h) {
    delete h;
    return AQ_OK;
}

int aq_last_cuda_error(aq_handle_t h) { return h ? h->last_cuda_error : 0; }
}  // extern "C"

namespace aq {
int handle_device(aq_handle_t h) { return h ? h->dev.device : -1; }
void handle_record_cuda_error(aq_handle_t h, cudaError_t e) {
    if (h) h->last_cuda_error = (int)e;
}
}  // namespace aq

extern "C" {

int aq_set_weights_stable(aq_handle_t h, int enabled) {
    if (!h) return AQ_ERR_INVALID_ARG;
    h->weights_stable = enabled ? 1 : 0;
    return AQ_OK;
}

int aq_set_kernel(aq_handle_t h, int kernel) {
    if (!h || kernel < AQ_KERNEL_AUTO || kernel > AQ_KERNEL_DECODE) return AQ_ERR_INVALID_ARG;
    h->kernel_choice = kernel;
    return AQ_OK;
}

size_t aq_packed_w4_bytes(int N, int K) {
    if (N < 1 || K < 32 || K % 32) return 0;
    return (size_t)round_up(N, kTileN) * (size_t)round_up(K, kTileK) / 2;
}

size_t aq_scales_bytes(int N, int K, int group_size) {
    if (N < 1 || K < 32 || K % 32 || (group_size != 0 && group_size != 128) || (group_size && K % 128)) return 0;
    const size_t G = group_size ? (size_t)K / 128 : 1;
    return G * (size_t)round_up(N, kTileN) * sizeof(__half);
}

size_t aq_workspace_bytes(int M, int K, int N, int group_size) {
    if (check_shape(M, K, N, group_size) != AQ_OK) return 0;
    return workspace_bytes(M, K, N, group_size);
}

size_t aq_workspace_min_bytes(int M, int K, int N, int group_size) {
    if (check_shape(M, K, N, group_size) != AQ_OK) return 0;
    return workspace_min_bytes(M, K, N);
}

int aq_pack_w4(aq_handle_t h, const void* w_fp16, int N, int K, int group_size, void* w_packed,
               void* w_scales, void* stream) {
    if (!h || !w_fp16 || !w_packed || !w_scales) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(1, K, N, group_size);
    if (s != AQ_OK) return s;
    if (!aligned(w_fp16, 16) || !aligned(w_packed, 16) || !aligned(w_scales, 2)) return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_pack_w4(static_cast<const __half*>(w_fp16), N, K, group_size,
                                         static_cast<uint8_t*>(w_packed), static_cast<__half*>(w_scales),
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_unpack_w4(aq_handle_t h, const void* w_packed, int N, int K, int8_t* codes, void* stream) {
    if (!h || !w_packed || !codes) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(1, K, N, 0);
    if (s != AQ_OK) return s;
    const cudaError_t e = launch_unpack_w4(static_cast<const uint8_t*>(w_packed), N, K, codes,
                                           static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

static int quantize_impl(aq_handle_t h, const void* x_fp16, int M, int K, int bits, int scale_mode,
                         int clip_shift_or_exp, const int32_t* row_idx, int8_t* q, int32_t* scale_exp_out,
                         void* workspace, size_t workspace_bytes_, void* stream_, const uint8_t* alpha, int k_max) {
    if (!h || !x_fp16 || !q) return AQ_ERR_INVALID_ARG;
    if (bits != 8 && bits != 4) return AQ_ERR_INVALID_ARG;
    if (scale_mode != AQ_SCALE_DYNAMIC && scale_mode != AQ_SCALE_STATIC) return AQ_ERR_INVALID_ARG;
    if (scale_mode == AQ_SCALE_DYNAMIC && (clip_shift_or_exp < 0 || clip_shift_or_exp > 16)) return AQ_ERR_INVALID_ARG;
    if (scale_mode == AQ_SCALE_STATIC && (clip_shift_or_exp < -40 || clip_shift_or_exp > 40)) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, 1, 0);
    if (s != AQ_OK) return s;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(x_fp16, 16) || !aligned(q, 16) || !aligned(workspace, 256) ||
        (scale_exp_out && !aligned(scale_exp_out, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    const __half* xh = static_cast<const __half*>(x_fp16);
    const cudaError_t e = quantize_dispatch(h, xh, M, K, row_idx, bits, scale_mode, clip_shift_or_exp, ctl, q,
                                            scale_exp_out, alpha, k_max, stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_quantize_act(aq_handle_t h, const void* x_fp16, int M, int K, int bits, int scale_mode,
                    int clip_shift_or_exp, const int32_t* row_idx, int8_t* q, int32_t* scale_exp_out,
                    void* workspace, size_t workspace_bytes_, void* stream) {
    return quantize_impl(h, x_fp16, M, K, bits, scale_mode, clip_shift_or_exp, row_idx, q, scale_exp_out, workspace,
                         workspace_bytes_, stream, nullptr, 0);
}

int aq_quantize_act_trip(aq_handle_t h, const void* x_fp16, int M, int K, const uint8_t* alpha, int k_max,
                         int scale_mode, int clip_shift_or_exp, const int32_t* row_idx, int8_t* q,
                         int32_t* scale_exp_out, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!trip_args_ok(alpha, k_max)) return AQ_ERR_INVALID_ARG;
    if (!aligned(alpha, 16)) return AQ_ERR_ALIGNMENT;
    return quantize_impl(h, x_fp16, M, K, 4, scale_mode, clip_shift_or_exp, row_idx, q, scale_exp_out, workspace,
                         workspace_bytes_, stream, alpha, k_max);
}

int aq_trip_calibrate(aq_handle_t h, const void* x_fp16, int M, int K, int k_max, const int32_t* row_idx,
                      uint8_t* alpha_out, int32_t* scale_exp_out, void* workspace, size_t workspace_bytes_,
                      void* stream_) {
    if (!h || !x_fp16 || !alpha_out || k_max < 0 || k_max > 4) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, 1, 0);
    if (s != AQ_OK) return s;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(x_fp16, 16) || !aligned(workspace, 256) || (scale_exp_out && !aligned(scale_exp_out, 4)) ||
        (row_idx && !aligned(row_idx, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    e = launch_trip_calibrate(static_cast<const __half*>(x_fp16), M, K, row_idx, 4, k_max, ctl, alpha_out,
                              scale_exp_out, h->dev, stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_linear_w4a4_trip(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                        const void* w_scales, int N, int group_size, const uint8_t* alpha, int k_max,
                        int scale_mode, int clip_shift_or_exp, const int32_t* row_idx, void* y_fp16,
                        int32_t* acc_dump, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!trip_args_ok(alpha, k_max)) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 4, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp,
                       row_idx, y_fp16, acc_dump, workspace, workspace_bytes_, stream, alpha, k_max);
}

int aq_linear_w4a8(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                   const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                   const int32_t* row_idx, void* y_fp16, int32_t* acc_dump, void* workspace,
                   size_t workspace_bytes_, void* stream) {
    return linear_impl(h, 8, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp,
                       row_idx, y_fp16, acc_dump, workspace, workspace_bytes_, stream);
}

int aq_linear_w4a4(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                   const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                   const int32_t* row_idx, void* y_fp16, int32_t* acc_dump, void* workspace,
                   size_t workspace_bytes_, void* stream) {
    return linear_impl(h, 4, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp,
                       row_idx, y_fp16, acc_dump, workspace, workspace_bytes_, stream);
}

int aq_gemm_w4(aq_handle_t h, const int8_t* q, int M, int K, const void* w_packed, const void* w_scales,
               int N, int group_size, const int32_t* scale_exp, void* y_fp16, int32_t* acc_dump,
               void* workspace, size_t workspace_bytes_, void* stream_) {
    if (!h || !q || !w_packed || !w_scales || !scale_exp || !y_fp16) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, N, group_size);
    if (s != AQ_OK) return s;
    if (!workspace || workspace_bytes_ < workspace_min_bytes(M, K, N)) return AQ_ERR_WORKSPACE;
    if (!aligned(q, 16) || !aligned(w_packed, 16) || !aligned(w_scales, 2) || !aligned(y_fp16, 2) ||
        !aligned(workspace, 256) || !aligned(scale_exp, 4) || (acc_dump && !aligned(acc_dump, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const Workspace w = carve(workspace, M, K, N, workspace_bytes_);
    if (kernel_for(h, M) == AQ_KERNEL_TENSOR) {       // the decode kernels clear the status word themselves
        const cudaError_t e = cudaMemsetAsync(w.ctl, 0, sizeof(Control), stream);
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    GemmArgs g;
    g.q = q; g.M = M; g.K = K; g.N = N; g.group = group_size;
    g.w_packed = static_cast<const uint8_t*>(w_packed);
    g.w_scales = static_cast<const __half*>(w_scales);
    g.scale_exp = scale_exp;
    g.y = static_cast<__half*>(y_fp16);
    g.acc_dump = acc_dump;
    g.ctl = w.ctl; g.scratch = w.scratch; g.scratch_bytes = w.scratch_bytes;
    g.split_scratch = w.split_scratch; g.split_bytes = w.split_bytes;
    return run_gemm(h, g, stream);
}

size_t aq_act4_bytes(int M, int K) {
    if (M < 1 || K < 32 || K % 32) return 0;
    return (size_t)M * (size_t)K / 2;
}

int aq_act4_pack(aq_handle_t h, const int8_t* q, int M, int K, void* q4, void* stream) {
    if (!h || !q || !q4) return AQ_ERR_INVALID_ARG;
    if (M < 1 || K < 32 || K % 32) return AQ_ERR_SHAPE;
    if (!aligned(q, 16) || !aligned(q4, 16)) return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_act4_pack(q, (size_t)M * K, static_cast<uint8_t*>(q4), static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_act4_unpack(aq_handle_t h, const void* q4, int M, int K, int8_t* q, void* stream) {
    if (!h || !q || !q4) return AQ_ERR_INVALID_ARG;
    if (M < 1 || K < 32 || K % 32) return AQ_ERR_SHAPE;
    if (!aligned(q, 16) || !aligned(q4, 16)) return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_act4_unpack(static_cast<const uint8_t*>(q4), (size_t)M * K, q, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_quantize_act4(aq_handle_t h, const void* x_fp16, int M, int K, int scale_mode, int clip_shift_or_exp,
                     const int32_t* row_idx, void* q4, int32_t* scale_exp_out, void* workspace,
                     size_t workspace_bytes_, void* stream) {
    if (!q4) return AQ_ERR_INVALID_ARG;
    if (!aligned(q4, 16)) return AQ_ERR_ALIGNMENT;
    if (M < 1 || K < 128 || K % 128) return AQ_ERR_SHAPE;
    // the codes pass through the workspace's code area in one-byte containers on their way to the nibbles
    if (!workspace || workspace_bytes_ < sizeof(Control) + up256((size_t)M * K)) return AQ_ERR_WORKSPACE;
    int8_t* codes = reinterpret_cast<int8_t*>(static_cast<uint8_t*>(workspace) + sizeof(Control));
    const int s = quantize_impl(h, x_fp16, M, K, 4, scale_mode, clip_shift_or_exp, row_idx, codes, scale_exp_out,
                                workspace, workspace_bytes_, stream, nullptr, 0);
    if (s != AQ_OK) return s;
    const cudaError_t e = launch_act4_pack(codes, (size_t)M * K, static_cast<uint8_t*>(q4), static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_gemm_w4_act4(aq_handle_t h, const void* q4, int M, int K, const void* w_packed, const void* w_scales,
                    int N, int group_size, const int32_t* scale_exp, void* y_fp16, int32_t* acc_dump,
                    void* workspace, size_t workspace_bytes_, void* stream_) {
    if (!h || !q4) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, N, group_size);
    if (s != AQ_OK) return s;
    if (!workspace || workspace_bytes_ < workspace_min_bytes(M, K, N)) return AQ_ERR_WORKSPACE;
    if (!aligned(q4, 16) || !aligned(workspace, 256)) return AQ_ERR_ALIGNMENT;
    const Workspace w = carve(workspace, M, K, N, workspace_bytes_);
    const cudaError_t e = launch_act4_unpack(static_cast<const uint8_t*>(q4), (size_t)M * K, w.codes,
                                             static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) return cuda_fail(h, e);
    return aq_gemm_w4(h, w.codes, M, K, w_packed, w_scales, N, group_size, scale_exp, y_fp16, acc_dump, workspace,
                      workspace_bytes_, stream_);
}

int aq_token_select(aq_handle_t h, const float* scores, int M, int n_keep, int32_t* idx, void* workspace,
                    size_t workspace_bytes_, void* stream) {
    if (!h || !scores || (!idx && n_keep > 0)) return AQ_ERR_INVALID_ARG;
    if (M < 1 || M > 65536 || n_keep < 0 || n_keep > M) return AQ_ERR_SHAPE;
    if (!workspace || workspace_bytes_ < sizeof(Control) + up256((size_t)M)) return AQ_ERR_WORKSPACE;
    if (!aligned(scores, 4) || !aligned(idx, 4) || !aligned(workspace, 256)) return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_token_select(scores, M, n_keep, idx,
                                              static_cast<uint8_t*>(workspace) + sizeof(Control),
                                              static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_token_compact(aq_handle_t h, const void* x_fp16, int M, int K, const int32_t* idx, int n_keep,
                     void* x_out, void* stream) {
    if (!h || !x_fp16 || !idx || !x_out) return AQ_ERR_INVALID_ARG;
    if (M < 1 || n_keep < 0 || n_keep > M || K < 8 || K % 8) return AQ_ERR_SHAPE;
    if (!aligned(x_fp16, 16) || !aligned(x_out, 16) || !aligned(idx, 4)) return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_token_compact(static_cast<const __half*>(x_fp16), K, idx, n_keep,
                                               static_cast<__half*>(x_out), h->dev,
                                               static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_weight_offsets(aq_handle_t h, const void* w_packed, const void* w_scales, int N, int K, int group_size,
                      float* r_out, void* stream) {
    if (!h || !w_packed || !w_scales || !r_out) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(1, K, N, group_size);
    if (s != AQ_OK) return s;
    if (!aligned(w_packed, 16) || !aligned(w_scales, 2) || !aligned(r_out, 4)) return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_weight_offsets(static_cast<const uint8_t*>(w_packed), static_cast<const __half*>(w_scales),
                                                N, K, group_size, r_out, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_quantize_act_asym(aq_handle_t h, const void* x_fp16, int M, int K, int bits, const int32_t* row_idx, int8_t* q,
                         int32_t* scale_exp_out, int32_t* zero_point_out, void* workspace, size_t workspace_bytes_,
                         void* stream_) {
    if (!h || !x_fp16 || !q || (bits != 8 && bits != 4)) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, 1, 0);
    if (s != AQ_OK) return s;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(x_fp16, 16) || !aligned(q, 16) || !aligned(workspace, 256) ||
        (scale_exp_out && !aligned(scale_exp_out, 4)) || (zero_point_out && !aligned(zero_point_out, 4)) ||
        (row_idx && !aligned(row_idx, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e == cudaSuccess)
        e = launch_quantize_asym(static_cast<const __half*>(x_fp16), M, K, row_idx, bits, ctl, q, scale_exp_out,
                                 zero_point_out, h->dev, stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_linear_w4a8_asym(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                        const float* w_offsets, int N, int group_size, const int32_t* row_idx, void* y_fp16,
                        int32_t* acc_dump, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!w_offsets) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 8, x_fp16, M, K, w_packed, w_scales, N, group_size, AQ_SCALE_DYNAMIC, 0, row_idx, y_fp16,
                       acc_dump, workspace, workspace_bytes_, stream, nullptr, 0, w_offsets);
}

int aq_linear_w4a4_asym(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                        const float* w_offsets, int N, int group_size, const int32_t* row_idx, void* y_fp16,
                        int32_t* acc_dump, void* workspace, size_t workspace_bytes_, void* stream) {
    if (!w_offsets) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 4, x_fp16, M, K, w_packed, w_scales, N, group_size, AQ_SCALE_DYNAMIC, 0, row_idx, y_fp16,
                       acc_dump, workspace, workspace_bytes_, stream, nullptr, 0, w_offsets);
}

int aq_linear_w4a8_chain(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                         int N, int group_size, int scale_mode, int clip_shift_or_exp, const int32_t* row_idx,
                         int8_t* q_next, int next_bits, int next_exp, int32_t* acc_dump, void* workspace,
                         size_t workspace_bytes_, void* stream) {
    if (!q_next) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 8, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp, row_idx,
                       nullptr, acc_dump, workspace, workspace_bytes_, stream, nullptr, 0, nullptr, q_next, next_bits,
                       next_exp);
}

int aq_linear_w4a4_chain(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                         int N, int group_size, int scale_mode, int clip_shift_or_exp, const int32_t* row_idx,
                         int8_t* q_next, int next_bits, int next_exp, int32_t* acc_dump, void* workspace,
                         size_t workspace_bytes_, void* stream) {
    if (!q_next) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 4, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp, row_idx,
                       nullptr, acc_dump, workspace, workspace_bytes_, stream, nullptr, 0, nullptr, q_next, next_bits,
                       next_exp);
}

int aq_linear_w4a8_chain_act4(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                              const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                              const int32_t* row_idx, void* q4_next, int next_exp, int32_t* acc_dump, void* workspace,
                              size_t workspace_bytes_, void* stream) {
    if (!q4_next) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 8, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp, row_idx,
                       nullptr, acc_dump, workspace, workspace_bytes_, stream, nullptr, 0, nullptr,
                       static_cast<int8_t*>(q4_next), 4, next_exp, true);
}

int aq_linear_w4a4_chain_act4(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                              const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                              const int32_t* row_idx, void* q4_next, int next_exp, int32_t* acc_dump, void* workspace,
                              size_t workspace_bytes_, void* stream) {
    if (!q4_next) return AQ_ERR_INVALID_ARG;
    return linear_impl(h, 4, x_fp16, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp, row_idx,
                       nullptr, acc_dump, workspace, workspace_bytes_, stream, nullptr, 0, nullptr,
                       static_cast<int8_t*>(q4_next), 4, next_exp, true);
}

int aq_log2_quantize(aq_handle_t h, const void* x_fp16, long long count, int bits, int8_t* codes,
                     uint32_t* max_bits_out, void* workspace, size_t workspace_bytes_, void* stream_) {
    if (!h || !x_fp16 || !codes || count < 1 || (bits != 8 && bits != 4)) return AQ_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(x_fp16, 2) || !aligned(workspace, 256) || (max_bits_out && !aligned(max_bits_out, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e == cudaSuccess)
        e = launch_log2_quantize(static_cast<const __half*>(x_fp16), count, bits, ctl, codes, max_bits_out, h->dev, stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_log2_quantize_factors(aq_handle_t h, const void* x_fp16, long long count, uint8_t* factors,
                             uint32_t* max_bits_out, void* workspace, size_t workspace_bytes_, void* stream_) {
    if (!h || !x_fp16 || !factors || count < 1) return AQ_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(x_fp16, 2) || !aligned(workspace, 256) || (max_bits_out && !aligned(max_bits_out, 4)))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e == cudaSuccess)
        e = launch_log2_quantize(static_cast<const __half*>(x_fp16), count, 4, ctl, reinterpret_cast<int8_t*>(factors),
                                 max_bits_out, h->dev, stream, true);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_attn_v_log2(aq_handle_t h, const int8_t* p_codes, const uint32_t* p_max_bits, const int8_t* v_codes,
                   const int32_t* v_scale_exp, int H, int M, int J, int D, int bits, void* y_fp16, int32_t* acc_dump,
                   void* stream) {
    if (!h || !p_codes || !p_max_bits || !v_codes || !v_scale_exp || !y_fp16) return AQ_ERR_INVALID_ARG;
    if (bits != 4) return AQ_ERR_INVALID_ARG;          // shifts up to kmax = 7; 8-bit codes would shift by up to 127
    if (H < 1 || M < 1 || J < 1 || J > 65536 || D < 4 || D > 1024 || D % 4 != 0 || 256 % (D / 4) != 0 || H > 65535)
        return AQ_ERR_SHAPE;
    if (!aligned(v_codes, 4) || !aligned(y_fp16, 2) || !aligned(p_max_bits, 4) || !aligned(v_scale_exp, 4) ||
        (acc_dump && !aligned(acc_dump, 4)))
        return AQ_ERR_ALIGNMENT;
    const cudaError_t e = launch_attn_v_log2(p_codes, p_max_bits, v_codes, v_scale_exp, H, M, J, D, bits,
                                             static_cast<__half*>(y_fp16), acc_dump, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

size_t aq_attn_workspace_bytes(int H, int M, int J, int D) {
    if (H < 1 || M < 1 || J < 1 || D < 1) return 0;
    return sizeof(Control) + attn_tc_scratch_bytes(H, M, J, D);
}

static int attn_v_tc_impl(aq_handle_t h, bool p_is_factors, const int8_t* p_codes, const uint32_t* p_max_bits, const int8_t* v_codes,
                      const int32_t* v_scale_exp, int H, int M, int J, int D, void* y_fp16, void* workspace,
                      size_t workspace_bytes_, void* stream_) {
    if (!h || !p_codes || !p_max_bits || !v_codes || !v_scale_exp || !y_fp16) return AQ_ERR_INVALID_ARG;
    if (H < 1 || H > 65535 || M < 1 || J < 16 || J > 65536 || J % 16 != 0 || (D != 64 && D != 128)) return AQ_ERR_SHAPE;
    if ((long long)H * M > 0x7FFFFFFFll || (long long)H * D > 0x7FFFFFFFll) return AQ_ERR_SHAPE;
    if (!workspace || workspace_bytes_ < aq_attn_workspace_bytes(H, M, J, D)) return AQ_ERR_WORKSPACE;
    if (!aligned(p_codes, p_is_factors ? 16 : 4) || !aligned(v_codes, 1) || !aligned(y_fp16, 16) || !aligned(p_max_bits, 4) ||
        !aligned(v_scale_exp, 4) || !aligned(workspace, 256))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e == cudaSuccess)
        e = launch_attn_v_log2_tc(p_codes, p_max_bits, v_codes, v_scale_exp, H, M, J, D, static_cast<__half*>(y_fp16), ctl,
                                  static_cast<uint8_t*>(workspace) + sizeof(Control), h->dev, stream, p_is_factors);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_attn_v_log2_tc(aq_handle_t h, const int8_t* p_codes, const uint32_t* p_max_bits, const int8_t* v_codes,
                      const int32_t* v_scale_exp, int H, int M, int J, int D, void* y_fp16, void* workspace,
                      size_t workspace_bytes_, void* stream_) {
    return attn_v_tc_impl(h, false, p_codes, p_max_bits, v_codes, v_scale_exp, H, M, J, D, y_fp16, workspace,
                          workspace_bytes_, stream_);
}

int aq_attn_v_factors_tc(aq_handle_t h, const uint8_t* p_factors, const uint32_t* p_max_bits, const int8_t* v_codes,
                         const int32_t* v_scale_exp, int H, int M, int J, int D, void* y_fp16, void* workspace,
                         size_t workspace_bytes_, void* stream_) {
    return attn_v_tc_impl(h, true, reinterpret_cast<const int8_t*>(p_factors), p_max_bits, v_codes, v_scale_exp, H, M, J, D,
                          y_fp16, workspace, workspace_bytes_, stream_);
}

int aq_attn_qk_tc(aq_handle_t h, const int8_t* q_codes, const int32_t* q_scale_exp, const int8_t* k_codes,
                  const int32_t* k_scale_exp, int H, int M, int J, int D, void* s_fp16, void* workspace,
                  size_t workspace_bytes_, void* stream_) {
    if (!h || !q_codes || !q_scale_exp || !k_codes || !k_scale_exp || !s_fp16) return AQ_ERR_INVALID_ARG;
    if (H < 1 || H > 65535 || M < 1 || J < 8 || J % 8 != 0 || D != 128) return AQ_ERR_SHAPE;
    if ((long long)H * M > 0x7FFFFFFFll || (long long)H * J > 0x7FFFFFFFll || (J + 127) / 128 > 65535) return AQ_ERR_SHAPE;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(q_codes, 16) || !aligned(k_codes, 16) || !aligned(s_fp16, 16) || !aligned(q_scale_exp, 4) ||
        !aligned(k_scale_exp, 4) || !aligned(workspace, 256))
        return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e == cudaSuccess)
        e = launch_attn_qk_tc(q_codes, q_scale_exp, k_codes, k_scale_exp, H, M, J, D, static_cast<__half*>(s_fp16), ctl,
                              h->dev, stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_prune_schedule(int M, double beta, int m, int32_t* n_keep_out, double* gamma_out) {
    if (M < 1 || m < 1 || !(beta >= 0.0) || !(beta < 1.0) || !n_keep_out) return AQ_ERR_INVALID_ARG;
    const double gamma = 1.0 - pow(1.0 - beta, 1.0 / (double)m);       // Eq. 9
    if (gamma_out) *gamma_out = gamma;
    int n = M;
    for (int i = 0; i < m; ++i) {
        const double kept = ceil((double)n * (1.0 - gamma) - 1e-9);       // the tolerance keeps exact products exact
        n = kept < 1.0 ? 1 : (int)kept;
        n_keep_out[i] = n;
    }
    return AQ_OK;
}

size_t aq_linear_host_scratch_bytes(int M, int K, int N, int group_size) {
    if (check_shape(M, K, N, group_size) != AQ_OK) return 0;
    return up256((size_t)M * K * 2) + up256((size_t)M * N * 2) + workspace_bytes(M, K, N, group_size);
}

static int linear_host_impl(aq_handle_t h, int bits, const void* x_host, int M, int K, const void* w_packed,
                            const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                            void* y_host, void* device_scratch, size_t scratch_bytes, void* stream_, bool wait) {
    if (!h || !x_host || !y_host) return AQ_ERR_INVALID_ARG;
    if (bits != 8 && bits != 4) return AQ_ERR_INVALID_ARG;
    const int s = check_shape(M, K, N, group_size);
    if (s != AQ_OK) return s;
    if (!device_scratch || scratch_bytes < aq_linear_host_scratch_bytes(M, K, N, group_size)) return AQ_ERR_WORKSPACE;
    if (!aligned(device_scratch, 256)) return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    uint8_t* b = static_cast<uint8_t*>(device_scratch);
    void* x_dev = b;
    void* y_dev = b + up256((size_t)M * K * 2);
    void* ws = b + up256((size_t)M * K * 2) + up256((size_t)M * N * 2);
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    const int rc = linear_impl(h, bits, x_dev, M, K, w_packed, w_scales, N, group_size, scale_mode,
                               clip_shift_or_exp, nullptr, y_dev, nullptr, ws, workspace_bytes(M, K, N, group_size), stream_);
    if (rc != AQ_OK) return rc;
    e = cudaMemcpyAsync(y_host, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if (!wait) return AQ_OK;
    e = cudaStreamSynchronize(stream);
    return e == cudaSuccess ? AQ_OK : cuda_fail(h, e);
}

int aq_linear_host(aq_handle_t h, int bits, const void* x_host, int M, int K, const void* w_packed,
                   const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                   void* y_host, void* device_scratch, size_t scratch_bytes, void* stream) {
    return linear_host_impl(h, bits, x_host, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp,
                            y_host, device_scratch, scratch_bytes, stream, true);
}

int aq_linear_host_async(aq_handle_t h, int bits, const void* x_host, int M, int K, const void* w_packed,
                         const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                         void* y_host, void* device_scratch, size_t scratch_bytes, void* stream) {
    return linear_host_impl(h, bits, x_host, M, K, w_packed, w_scales, N, group_size, scale_mode, clip_shift_or_exp,
                            y_host, device_scratch, scratch_bytes, stream, false);
}

int aq_probe_int8_mma(aq_handle_t h, int iters, int a_from_tmem, double* ops_out, void* workspace,
                      size_t workspace_bytes_, void* stream_) {
    if (!h || iters < 1 || iters > (1 << 24)) return AQ_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes_ < sizeof(Control)) return AQ_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return AQ_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Control* ctl = static_cast<Control*>(workspace);
    cudaError_t e = cudaMemsetAsync(ctl, 0, sizeof(Control), stream);
    if (e == cudaSuccess) e = launch_int8_probe(iters, a_from_tmem ? 1 : 0, ctl, h->dev, stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if (ops_out) *ops_out = 2.0 * 128.0 * 256.0 * 32.0 * 4.0 * (double)iters * (double)h->dev.sm_count;
    return AQ_OK;
}

int aq_check_workspace(aq_handle_t h, const void* workspace, void* stream_) {
    if (!h || !workspace) return AQ_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(h, e);
    Control c;
    e = cudaMemcpy(&c, workspace, sizeof(Control), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if (c.status == 11u) return AQ_ERR_INVALID_ARG;     // aq_attn_v_log2_tc met a negative code
    return c.status ? AQ_ERR_DEVICE_TIMEOUT : AQ_OK;
}

}  // extern "C"

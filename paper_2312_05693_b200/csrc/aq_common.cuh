// Shared declarations for the agileq kernels (device-side helpers, layout constants,
// the workspace control block and the launcher prototypes).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>

#include "../../include/agileq.h"

namespace aq {

// ---------------------------------------------------------------------------------------
// Packed 4-bit weight layout (device-native; defined only here and in aq_pack.cu).
//
// Rows are padded to Npad = ceil(N/128)*128. The matrix is cut into blocks of 128 rows x
// 128 k. Block (nt, kb) starts at byte ((nt * K/128 + kb) * 8192). Inside a block, the
// 16-byte unit (j, r), j = 0..3, r = 0..127, sits at byte (j*128 + r)*16 and holds the 32
// codes k = kb*128 + 32j .. +31 of row nt*128 + r. Inside a unit, byte b of 32-bit word i
// (i = 0..3, little endian) holds code k0+b in its low nibble and code k0+4+b in its high
// nibble, k0 = kb*128 + 32j + 8i, as two's-complement nibbles.
//
// Why: a warp reads 512 contiguous bytes per load; "(w << 4) & 0xF0F0F0F0" and
// "w & 0xF0F0F0F0" turn one word into two words of four int8 values equal to 16*code in k
// order, with no sign extension. Integer sums therefore come out multiplied by 16 and are
// shifted right by 4 (exact) before use.
// ---------------------------------------------------------------------------------------
constexpr int kTileN = 128;          // rows per packed block
constexpr int kTileK = 128;          // k per packed block (= the weight-scale group)
constexpr int kBlockBytes = kTileN * kTileK / 2;   // 8192

__host__ __device__ inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
// Blocks of 128 k that cover K. With one scale per channel K need only be a multiple of 32: the last
// block is then padded with zero codes at pack time, so whatever the activation side delivers for
// k >= K (zeros from a tensor map's bounds, or stale staging bytes) contributes nothing.
__host__ __device__ inline int k_blocks(int K) { return (K + kTileK - 1) / kTileK; }
__host__ __device__ inline size_t packed_unit_offset(int KB, int nt, int kb, int j, int r) {
    return ((size_t)nt * KB + kb) * kBlockBytes + (size_t)(j * kTileN + r) * 16;
}

// ---------------------------------------------------------------------------------------
// Workspace layout: [control block 256 B][activation codes M*K int8, padded to 256 B]
// [kernel scratch].
// ---------------------------------------------------------------------------------------
struct Control {
    unsigned int absmax_bits;   // fp16 bit pattern of max|x| (atomicMax target), cleared per call
    int scale_exp;              // layer exponent e
    unsigned int status;        // non-zero: a bounded wait gave up
    unsigned int counter;       // scratch counter
    unsigned int min_key, max_key;   // zero-point variant: order-preserving keys of min(x), max(x)
    int zero_point;             // zero-point variant: zp of Eq. 7
    unsigned int split_flags[57];   // tensor kernel: one bit per (shared tile, epilogue warp), "first half arrived"
    static constexpr int kMaxSplitTiles = 57 * 32 / 12;   // up to twelve epilogue warps per tile
};
static_assert(sizeof(Control) == 256, "control block is 256 bytes");

// Layer exponent from max|x| (fp16 bits): the smallest e with qmax * 2^e >= a, qmax =
// 2^(bits-1)-1 (Eq. 6 read as a symmetric power-of-two scale). Uses the binary expansion
// a = m * 2^ex, m in [0.5, 1): qmax = mq * 2^xq with mq = 127/128 (xq = 7) or 7/8 (xq = 3),
// so e = ex - xq, plus one if m > mq. a == 0 gives 0; +Inf counts as 65504.
__device__ inline int layer_exponent_from_bits(unsigned int absmax_bits, int bits) {
    unsigned int hb = absmax_bits & 0x7FFFu;
    if (hb == 0) return 0;
    if (hb >= 0x7C00u) hb = 0x7BFFu;
    const float a = __half2float(__ushort_as_half((unsigned short)hb));
    int ex;
    const float m = frexpf(a, &ex);
    const float mq = bits == 8 ? 0.9921875f : 0.875f;
    const int xq = bits == 8 ? 7 : 3;
    return ex - xq + (m > mq ? 1 : 0);
}

// ---------------------------------------------------------------------------------------
// Launchers (implemented one per .cu file). All enqueue on `stream` and return the CUDA
// launch status.
// ---------------------------------------------------------------------------------------
struct DeviceInfo {
    int device;
    int sm_count;
    int cc_major, cc_minor;
    size_t smem_optin;
    void* encode_tiled;   // cuTensorMapEncodeTiled, resolved through the runtime
};

// Opting a kernel in to more than 48 KB of dynamic shared memory acts on the current device only, so
// the "already done" flag is kept per device (a process may hold handles on several GPUs). One
// static instance per kernel, owned by that kernel's launcher.
constexpr int kMaxDevices = 64;
struct SmemOptIn {
    std::atomic<bool> done[kMaxDevices];
    template <class Kernel>
    cudaError_t ensure(Kernel kernel, int device, size_t bytes) {
        if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
        if (done[device].load(std::memory_order_acquire)) return cudaSuccess;
        const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e == cudaSuccess) done[device].store(true, std::memory_order_release);
        return e;
    }
};

cudaError_t launch_pack_w4(const __half* w, int N, int K, int group, uint8_t* packed, __half* scales,
                           cudaStream_t stream);
cudaError_t launch_unpack_w4(const uint8_t* packed, int N, int K, int8_t* codes, cudaStream_t stream);
// 4-bit activation codes, two per byte (code 2j in the low nibble of byte j); count = number of codes, a
// multiple of 16, both buffers 16-byte (codes) / 8-byte (packed) aligned.
cudaError_t launch_act4_pack(const int8_t* q, size_t count, uint8_t* out, cudaStream_t stream);
cudaError_t launch_act4_unpack(const uint8_t* packed, size_t count, int8_t* q, cudaStream_t stream);

cudaError_t launch_quantize(const __half* x, int M, int K, const int32_t* row_idx, int bits,
                            int scale_mode, int clip_shift_or_exp, Control* ctl, int8_t* q,
                            int32_t* scale_exp_out, const DeviceInfo& dev, cudaStream_t stream,
                            const uint8_t* alpha = nullptr, int k_max = 0);

// Activations of at most 262144 elements: one kernel that also initialises the control block.
bool quantize_small_fits(int M, int K);
cudaError_t launch_quantize_small(const __half* x, int M, int K, const int32_t* row_idx, int bits, int scale_mode,
                                  int clip_shift_or_exp, Control* ctl, int8_t* q, int32_t* scale_exp_out,
                                  cudaStream_t stream, const uint8_t* alpha = nullptr, int k_max = 0,
                                  bool early_dependents = false);

// Dynamic scale, any size: one cooperative kernel (absmax, exponent, codes). The control block must
// have been cleared (absmax_bits, counter) on the same stream before.
cudaError_t launch_quantize_fused(const __half* x, int M, int K, const int32_t* row_idx, int bits, int clip_shift,
                                  Control* ctl, int8_t* q, int32_t* scale_exp_out, const DeviceInfo& dev,
                                  cudaStream_t stream, const uint8_t* alpha = nullptr, int k_max = 0);
// TRIP factors (Eq. 5-8): `alpha` above is NULL or K bytes (16-byte aligned), one factor 0..k_max per
// input channel: channel k is quantized with the step 2^(e + alpha_k), its code stored shifted left by
// alpha_k, and the dynamic exponent is lowered by k_max (Eq. 6). The search of Eq. 8:
cudaError_t launch_trip_calibrate(const __half* x, int M, int K, const int32_t* row_idx, int bits, int k_max,
                                  Control* ctl, uint8_t* alpha_out, int32_t* scale_exp_out, const DeviceInfo& dev,
                                  cudaStream_t stream);

// Zero-point variant (Eq. 2, Eq. 5-7 with alpha = 0 and a power-of-two scale): one cooperative kernel
// finds minimum and maximum, then e, zp and the codes, stored as q - 2^(b-1) in int8. The control block
// must have been cleared.
cudaError_t launch_quantize_asym(const __half* x, int M, int K, const int32_t* row_idx, int bits, Control* ctl,
                                 int8_t* q, int32_t* scale_exp_out, int32_t* zero_point_out, const DeviceInfo& dev,
                                 cudaStream_t stream);
// r[n] = sum_g s_w[n,g] * sum_{k in g} c[n,k], from the packed weights (float [N]).
cudaError_t launch_weight_offsets(const uint8_t* packed, const __half* scales, int N, int K, int group, float* r,
                                  cudaStream_t stream);
// off[n] = -(zp - 2^(b-1)) * r[n] with zp from the control block.
cudaError_t launch_chan_offsets(const float* r, int N, int bits, const Control* ctl, float* off, cudaStream_t stream);

// Log2 codes of Eq. 3 (two kernels: layer maximum, codes) and attention x value on them (aq_attn.cu).
cudaError_t launch_log2_quantize(const __half* x, long long count, int bits, Control* ctl, int8_t* codes,
                                 uint32_t* max_bits_out, const DeviceInfo& dev, cudaStream_t stream, bool as_factors = false);
// The same product on the tensor cores, for non-negative P; scratch holds attn_tc_scratch_bytes().
size_t attn_tc_scratch_bytes(int H, int M, int J, int D);
cudaError_t launch_attn_v_log2_tc(const int8_t* pcodes, const uint32_t* max_bits, const int8_t* vq, const int32_t* e_v,
                                  int H, int M, int J, int D, __half* y, Control* ctl, void* scratch,
                                  const DeviceInfo& dev, cudaStream_t stream, bool p_is_factors = false);
// Query x key product on int8 codes (head dimension 128), same tensor-core kernel.
cudaError_t launch_attn_qk_tc(const int8_t* qc, const int32_t* e_q, const int8_t* kc, const int32_t* e_k, int H, int M,
                              int J, int D, __half* s_out, Control* ctl, const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_attn_v_log2(const int8_t* pcodes, const uint32_t* max_bits, const int8_t* vq, const int32_t* e_v,
                               int H, int M, int J, int D, int bits, __half* y, int32_t* acc_dump, cudaStream_t stream);

cudaError_t launch_token_select(const float* scores, int M, int n_keep, int32_t* idx, void* scratch,
                                cudaStream_t stream);
cudaError_t launch_token_compact(const __half* x, int K, const int32_t* idx, int n_keep, __half* out,
                                 const DeviceInfo& dev, cudaStream_t stream);

// Integer product + floating-point output on quantized codes.
struct GemmArgs {
    const int8_t* q;        // [M][K]
    int M, K, N, group;     // group: 0 or 128
    const uint8_t* w_packed;
    const __half* w_scales; // [G][Npad]
    const int32_t* scale_exp;
    __half* y;              // [M][N]
    int32_t* acc_dump;      // NULL or [M][N][G]
    Control* ctl;
    const float* chan_offset = nullptr;   // NULL or [N]: added to sum_g s*acc before the 2^e factor (zero-point term)
    // Chaining: when q_next is given the kernels write, instead of y, the next layer's activation codes
    // [M][N] int8: clip(round(y16 / 2^next_exp), -2^(b-1), 2^(b-1)-1), y16 the fp16 value y would have held.
    int8_t* q_next = nullptr;
    int next_bits = 8, next_exp = 0;
    // the next layer's 4-bit codes leave packed, two per byte [M][N/2] (code 2j in the low nibble of byte j);
    // needs next_bits == 4, N % 32 == 0 and a 16-byte aligned q_next
    bool next_packed = false;
    // The launch directly before this one on the stream is this call's own quantize (or offset) kernel: the
    // status word is already initialised, and the product kernels may be set up (the few-row streaming
    // kernel also starts streaming weights) while that kernel still runs (programmatic dependent launch;
    // they wait for that grid before they touch the codes). Weights cannot be in flight then: the quantize
    // kernels allow the dependent launch only once everything before them on the stream has completed (the
    // cooperative one is launched normally, the small one signals after its own wait for the kernel ahead).
    bool after_quantize = false;
    // The caller's promise (aq_set_weights_stable) that nothing in flight on the stream writes the packed
    // weights or their scales: the few-row kernel then allows the launch behind it at its very start and puts
    // its own first ring of weight copies in flight before it waits for the kernel ahead of it.
    bool weights_stable = false;
    // fp32 partial outputs of tiles whose k range two CTAs share (tensor kernel, per-group scales)
    float* split_scratch = nullptr;
    size_t split_bytes = 0;
    // One row (M = 1): the few-row streaming kernel quantizes the activations itself (no quantize kernel runs
    // ahead); q then receives the codes, the control block the exponent.
    const __half* fuse_x = nullptr;
    const int32_t* fuse_row_idx = nullptr;
    int fuse_bits = 8, fuse_scale_mode = 0, fuse_clip_shift_or_exp = 0;
    void* scratch;          // beyond control block + codes
    size_t scratch_bytes;
};
// Small accessors for code outside aq_api.cu that is handed a handle.
int handle_device(aq_handle_t h);
void handle_record_cuda_error(aq_handle_t h, cudaError_t e);

cudaError_t launch_gemm_tensor(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream);
// One scale per channel on tiles of 256 channels x 128 tokens (aq_gemm_wide.cu), for shapes it applies to.
bool gemm_wide_applies(const GemmArgs& a);
cudaError_t launch_gemm_wide(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream);
// Bytes of split_scratch the tensor kernel can use for these sizes on a GPU with sm_count SMs (0: none).
size_t tensor_split_scratch_bytes(int M, int K, int N, int group, int sm_count);
// Tensor-core rate probe: every SM issues iters x 4 MMAs of 128 x 256 x 32 (int8) on resident operands.
cudaError_t launch_int8_probe(int iters, int a_from_tmem, Control* ctl, const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_gemm_decode(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream);
bool decode_can_fuse_quantize(int M, int K, int N, int group, int sm_count);

}  // namespace aq

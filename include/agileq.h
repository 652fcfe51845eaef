/*
 * agileq: the quantized linear layer of Agile-Quant (arXiv 2312.05693) for NVIDIA B200
 * (sm_100a). C ABI, plain pointers and sizes.
 *
 * What the layer computes (paper Sec. 4.4, "Efficient TRIP Matrix Multiplication"):
 * activations are quantized layer-wise (one scale for the whole matrix), weights per
 * output channel (optionally per 128-wide group along K), products are summed as
 * integers and the sums are mapped back to floating point:
 *
 *     e    = layer exponent, scale 2^e               (Eq. 6, symmetric, alpha = 0)
 *     q    = clip(round(x / 2^e), -2^(b-1), 2^(b-1)-1)      (Eq. 1, Eq. 2 / Eq. 5, zp = 0)
 *     acc  = sum_k q[m,k] * c[n,k]                   (int32; Sec. 4.4, Algorithm 1)
 *     y    = fp16( 2^e * sum_g s_w[n,g] * acc[m,n,g] )
 *
 * Conventions
 *  - Every tensor pointer is a DEVICE pointer owned by the caller unless its name ends
 *    in "_host". The library never allocates or frees device memory; scratch comes from
 *    a caller-provided workspace. Pointers must be 16-byte aligned (256 for workspaces).
 *  - Calls enqueue work on the CUDA stream passed as `stream` (a cudaStream_t cast to
 *    void*, NULL = default stream) and return without synchronizing, except the calls
 *    documented as synchronizing.
 *  - Return value: AQ_OK (0) or a negative aq_status. On error nothing was enqueued.
 *  - Shapes: K % 32 == 0, 32 <= K <= 65536, and K % 128 == 0 when group_size is 128; N >= 1;
 *    M >= 1. group_size is 0 (one scale per output channel) or 128. Activation bits is 8 or 4
 *    (4-bit codes are stored one per int8, values -8..7).
 *  - Rounding is to nearest, ties to even.
 *  - Requires a device of compute capability 10.0 (B200); anything else is refused with
 *    AQ_ERR_UNSUPPORTED_DEVICE. There is no CPU or other fallback.
 */
#ifndef AGILEQ_H_
#define AGILEQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aq_context* aq_handle_t;

typedef enum aq_status {
    AQ_OK = 0,
    AQ_ERR_INVALID_ARG = -1,        /* NULL pointer, bad enum value, bad bit width */
    AQ_ERR_SHAPE = -2,              /* unsupported M / K / N / group_size / n_keep */
    AQ_ERR_ALIGNMENT = -3,          /* a pointer is not aligned as required */
    AQ_ERR_WORKSPACE = -4,          /* workspace NULL or smaller than aq_workspace_bytes() */
    AQ_ERR_UNSUPPORTED_DEVICE = -5, /* not compute capability 10.0 */
    AQ_ERR_CUDA = -6,               /* a CUDA call failed; see aq_last_cuda_error() */
    AQ_ERR_DEVICE_TIMEOUT = -7,     /* a bounded wait inside a kernel gave up */
    AQ_ERR_TOO_LARGE = -8           /* the sizes need more than the library's built-in scratch */
} aq_status;

/* How the layer exponent e is chosen (paper Eq. 6 read as a symmetric power-of-two
 * scale). DYNAMIC: e0 = smallest integer with (2^(b-1)-1) * 2^e0 >= max|x| over the rows
 * used, e = e0 - clip_shift (clip_shift >= 0 lets outliers saturate). STATIC: e is given. */
enum { AQ_SCALE_DYNAMIC = 0, AQ_SCALE_STATIC = 1 };

/* Which matrix-product kernel aq_linear_* / aq_gemm_w4 uses. AUTO picks the decode kernel
 * for M <= 16 and the tensor-core kernel otherwise; the others force one (for tests and
 * measurements). All give identical integer sums. */
enum { AQ_KERNEL_AUTO = 0, AQ_KERNEL_TENSOR = 1, AQ_KERNEL_DECODE = 2 };

const char* aq_status_string(int status);
int aq_version(void);

/* Handle: host-side state only (device properties, driver entry points). `device` is a
 * CUDA device ordinal; it must be the current device whenever the handle is used. */
int aq_create(aq_handle_t* out, int device);
int aq_destroy(aq_handle_t h);
/* The cudaError_t value of the last failed CUDA call made through this handle. */
int aq_last_cuda_error(aq_handle_t h);
/* Force a kernel choice for subsequent calls on this handle (AQ_KERNEL_*). */
int aq_set_kernel(aq_handle_t h, int kernel);
/* A scheduling promise, not part of the paper's method; off by default. enabled != 0 tells the library that,
 * for every later call on this handle, no work still in flight on the call's stream when the call is enqueued
 * writes the packed weights or weight scales the call reads (the usual case: weights are packed once, before
 * inference starts). The few-row kernels (M <= 16, one scale per channel) then let the launch behind them be
 * set up from their start and fetch their first 64 KB of weights per CTA before they wait for the kernel ahead
 * of them; everything else a call reads or writes still waits for that kernel. Results are the same bit for
 * bit; consecutive few-row calls on one stream overlap by a microsecond or two. With the promise broken (a
 * kernel that writes the weights is still running when the call starts) the call may read stale weights. */
int aq_set_weights_stable(aq_handle_t h, int enabled);

/* ---- sizes -------------------------------------------------------------------------- */
/* Bytes of the packed 4-bit weight buffer (rows are padded to a multiple of 128 channels, and K to a
 * multiple of 128 with zero codes; the size does not depend on group_size). */
size_t aq_packed_w4_bytes(int N, int K);
/* Version of the packed layout that aq_pack_w4 of this library writes. The packed buffer is a bare
 * array of blocks without a header, so a program that stores packed weights (a file, a cache) keeps
 * this number beside them and repacks when a later library reports another one. */
int aq_packed_w4_layout_version(void);
/* Bytes of the fp16 scale buffer: [G][Npad], G = 1 (group_size 0) or K/128, Npad = N
 * rounded up to 128; element (g, n) at index g*Npad + n. */
size_t aq_scales_bytes(int N, int K, int group_size);
/* Bytes of scratch that aq_quantize_act / aq_linear_* / aq_gemm_w4 / aq_token_select should get
 * for these sizes (M = rows actually multiplied). Always a multiple of 256. */
size_t aq_workspace_bytes(int M, int K, int N, int group_size);
/* The least the calls accept: control block, activation codes, per-row scratch, per-channel terms.
 * aq_workspace_bytes() adds, for per-group scales, room for the partial sums of output tiles whose
 * k range CTAs share; with less than that the kernel shares no tile (slower on some shapes; outputs
 * may then differ in the last fp32 rounding before the fp16 one, integer sums never). */
size_t aq_workspace_min_bytes(int M, int K, int N, int group_size);

/* ---- weights (offline; paper Sec. 4.4 last paragraph, Sec. 5.1: 4-bit per-channel weights)
 * Round-to-nearest symmetric quantization of w_fp16 [N,K] row-major:
 *   a = max|w| over the channel (or 128-wide group), s = fp16(a/7) (1 if a == 0, the
 *   smallest positive fp16 if a/7 underflows), c = clip(round(w/s), -8, 7).
 * Writes the codes in the library's device-native packed layout (opaque; read it back
 * with aq_unpack_w4) and the scales as described at aq_scales_bytes(). Weights must be
 * finite. */
int aq_pack_w4(aq_handle_t h, const void* w_fp16, int N, int K, int group_size,
               void* w_packed, void* w_scales, void* stream);
/* Test utility: packed layout -> int8 codes [N,K] row-major. */
int aq_unpack_w4(aq_handle_t h, const void* w_packed, int N, int K, int8_t* codes, void* stream);

/* ---- activations (paper Eq. 1, Eq. 2 / Eq. 5 with zp = 0; layer-wise scale, Sec. 4.4)
 * x_fp16 [M_in,K] row-major. row_idx == NULL: rows 0..M-1 are quantized; otherwise row
 * row_idx[i] (i < M) is read, so pruned tokens (Eq. 4) never enter the scale or the codes.
 * q [M,K] int8 row-major. scale_exp_out: one int32 on the device, receives e.
 * bits 8 or 4. NaN -> code 0 and is ignored by the scale; +-Inf saturate. */
int aq_quantize_act(aq_handle_t h, const void* x_fp16, int M, int K, int bits, int scale_mode,
                    int clip_shift_or_exp, const int32_t* row_idx, int8_t* q,
                    int32_t* scale_exp_out, void* workspace, size_t workspace_bytes,
                    void* stream);

/* ---- the layer (paper Sec. 4.4): quantize, integer product, floating-point output
 * y_fp16 [M,N] row-major. acc_dump: NULL, or int32 [M][N][G] (G as in aq_scales_bytes)
 * receiving the integer sums (test aid; slows the call). row_idx as above. */
int aq_linear_w4a8(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                   const void* w_scales, int N, int group_size, int scale_mode,
                   int clip_shift_or_exp, const int32_t* row_idx, void* y_fp16,
                   int32_t* acc_dump, void* workspace, size_t workspace_bytes, void* stream);
/* Same with 4-bit activation codes (paper Sec. 4.2: some activations take 4 bits). */
int aq_linear_w4a4(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                   const void* w_scales, int N, int group_size, int scale_mode,
                   int clip_shift_or_exp, const int32_t* row_idx, void* y_fp16,
                   int32_t* acc_dump, void* workspace, size_t workspace_bytes, void* stream);

/* The product and output steps alone, on codes q [M,K] that are already quantized;
 * scale_exp: device int32 holding e. */
int aq_gemm_w4(aq_handle_t h, const int8_t* q, int M, int K, const void* w_packed,
               const void* w_scales, int N, int group_size, const int32_t* scale_exp,
               void* y_fp16, int32_t* acc_dump, void* workspace, size_t workspace_bytes,
               void* stream);

/* ---- token pruning (paper Eq. 4: X^P = F^P(X), n < m tokens kept by importance)
 * aq_token_select: idx [n_keep] = indices of the n_keep largest scores, equal scores
 * resolved toward the lower index, in ascending order. scores fp32 [M], no NaN,
 * M <= 65536. aq_token_compact: x_out[i,:] = x[idx[i],:] (fp16 rows of K). */
int aq_token_select(aq_handle_t h, const float* scores, int M, int n_keep, int32_t* idx,
                    void* workspace, size_t workspace_bytes, void* stream);
int aq_token_compact(aq_handle_t h, const void* x_fp16, int M, int K, const int32_t* idx,
                     int n_keep, void* x_out, void* stream);

/* ---- per-channel TRIP factors (paper Eq. 5-8; Sec. 4.4 "Efficient TRIP Matrix Multiplication")
 * alpha: K bytes on the device (16-byte aligned), one factor per input channel, each in
 * 0..k_max, k_max <= 4. Channel k is quantized to a 4-bit code with the coarser step
 * 2^(e + alpha_k) (Eq. 5), and the code enters the integer product shifted left by alpha_k,
 * which is Sec. 4.4's move of the factor from the activation scale onto the weights (a 4-bit code
 * shifted by at most 4 still fits the int8 operand). The dynamic base exponent is
 * e = e0 - k_max - clip_shift, e0 the plain 4-bit layer exponent (Eq. 6 read as
 * s = 2^(e0 - K)), so channels with the largest factor still reach the layer maximum; in
 * static mode e is given. Outputs are y = 2^e * sum_g s_w[n,g] * acc[m,n,g] as before.
 * Factors above 4 are the caller's error (the shifted code would leave int8).
 *
 * aq_trip_calibrate: Eq. 8 with the clipping of Eq. 5: for every channel the factor in
 * 0..k_max with the least squared reconstruction error over the M calibration rows (kept
 * rows when row_idx is given), the smallest factor among equals; errors are summed in
 * binary64 over rows in ascending order. Writes alpha_out[K] and the base exponent
 * e = e0 - k_max of the calibration set. Non-finite values are skipped. */
int aq_trip_calibrate(aq_handle_t h, const void* x_fp16, int M, int K, int k_max, const int32_t* row_idx,
                      uint8_t* alpha_out, int32_t* scale_exp_out, void* workspace, size_t workspace_bytes,
                      void* stream);
/* As aq_quantize_act with bits = 4: q[m,k] = code * 2^alpha_k (int8). */
int aq_quantize_act_trip(aq_handle_t h, const void* x_fp16, int M, int K, const uint8_t* alpha, int k_max,
                         int scale_mode, int clip_shift_or_exp, const int32_t* row_idx, int8_t* q,
                         int32_t* scale_exp_out, void* workspace, size_t workspace_bytes, void* stream);
/* As aq_linear_w4a4 with the factors applied in the quantize step; the product kernels are unchanged. */
int aq_linear_w4a4_trip(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                        const void* w_scales, int N, int group_size, const uint8_t* alpha, int k_max,
                        int scale_mode, int clip_shift_or_exp, const int32_t* row_idx, void* y_fp16,
                        int32_t* acc_dump, void* workspace, size_t workspace_bytes, void* stream);

/* ---- activations with a zero point (paper Eq. 2, Eq. 5-7 with alpha = 0)
 * Unsigned codes q = CLIP(round(x / s) + zp, 0, 2^b - 1), zp = CLIP(round(-min / s), 0, 2^b - 1), with
 * the scale a power of two as everywhere here: s = 2^e, e the smallest integer with
 * (2^b - 1) * 2^e >= max - min over the (kept) activations; the range is widened to contain 0. NaN
 * is ignored by min / max and gets the code zp (value 0); +-Inf count as +-65504. The codes are
 * stored as q - 2^(b-1) in int8, and the layer is
 *   y[m,n] = fp16( 2^e * sum_g s_w[n,g] * sum_{k in g} (q[m,k] - zp) * c[n,k] ),
 * computed as the signed integer product plus the per-channel term -(zp - 2^(b-1)) * r[n], with
 * r[n] = sum_g s_w[n,g] * sum_{k in g} c[n,k] made once per weight matrix by aq_weight_offsets
 * (float [N] on the device). acc_dump, when given, receives the signed product
 * sum_{k in g} (q[m,k] - 2^(b-1)) * c[n,k] (the zero-point term is not in it). The scale is always
 * dynamic. */
int aq_weight_offsets(aq_handle_t h, const void* w_packed, const void* w_scales, int N, int K, int group_size,
                      float* r_out, void* stream);
int aq_quantize_act_asym(aq_handle_t h, const void* x_fp16, int M, int K, int bits, const int32_t* row_idx,
                         int8_t* q, int32_t* scale_exp_out, int32_t* zero_point_out, void* workspace,
                         size_t workspace_bytes, void* stream);
int aq_linear_w4a8_asym(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                        const float* w_offsets, int N, int group_size, const int32_t* row_idx, void* y_fp16,
                        int32_t* acc_dump, void* workspace, size_t workspace_bytes, void* stream);
int aq_linear_w4a4_asym(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                        const float* w_offsets, int N, int group_size, const int32_t* row_idx, void* y_fp16,
                        int32_t* acc_dump, void* workspace, size_t workspace_bytes, void* stream);

/* ---- chaining two layers (paper Sec. 4.4: the kernel's outputs are quantized back for the next
 * operation instead of leaving as floating point)
 * As aq_linear_w4a8 / aq_linear_w4a4, but instead of the fp16 outputs the call writes the NEXT layer's
 * activation codes q_next [M,N] int8 row-major: q_next = clip(round(y16 / 2^next_exp), -2^(b-1),
 * 2^(b-1)-1) with b = next_bits (8 or 4), where y16 is exactly the fp16 value the plain call would have
 * written (so the codes equal aq_quantize_act of that output with the static exponent next_exp; NaN -> 0).
 * The next layer then runs on the codes with aq_gemm_w4 (its scale_exp = next_exp on the device). The
 * exponent has to be known beforehand (calibration), since a layer-wide maximum of y does not exist
 * before the layer has finished. -40 <= next_exp <= 40. */
int aq_linear_w4a8_chain(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                         int N, int group_size, int scale_mode, int clip_shift_or_exp, const int32_t* row_idx,
                         int8_t* q_next, int next_bits, int next_exp, int32_t* acc_dump, void* workspace,
                         size_t workspace_bytes, void* stream);
int aq_linear_w4a4_chain(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed, const void* w_scales,
                         int N, int group_size, int scale_mode, int clip_shift_or_exp, const int32_t* row_idx,
                         int8_t* q_next, int next_bits, int next_exp, int32_t* acc_dump, void* workspace,
                         size_t workspace_bytes, void* stream);

/* ---- packed storage of 4-bit activation codes (paper Sec. 4.4: two adjacent 4-bit values share a
 * byte, as the weights do)
 * q4 [M, K/2] bytes, row-major, device: byte j of a row holds code 2j in bits 0-3 and code 2j+1 in
 * bits 4-7, two's-complement nibbles. K % 32 == 0; q and q4 16-byte aligned; aq_act4_bytes = M*K/2
 * (0 for sizes the calls reject).
 * aq_act4_pack: q int8 [M,K] with values in [-8, 7] (only the low four bits of each are kept).
 * aq_act4_unpack: the inverse, sign-extended int8 codes.
 * aq_quantize_act4: aq_quantize_act with bits = 4 whose codes are written packed; K % 128 == 0; the
 *   workspace must hold aq_workspace_bytes(M, K, 1, 0) (the codes pass through it in one-byte containers).
 * aq_gemm_w4_act4: aq_gemm_w4 on packed codes. The tensor cores have no 4-bit integer operand, so the
 *   codes are widened into the workspace's code area by one extra pass (M*K/2 bytes read, M*K written)
 *   before the product; what the packed form halves is the storage and traffic between layers.
 * aq_linear_w4a8_chain_act4 / aq_linear_w4a4_chain_act4: the chained calls above with next_bits = 4 whose
 *   codes leave the product kernels' epilogue already packed, q4_next [M, N/2]: no one-byte containers
 *   are written between the two layers. N % 32 == 0 (else AQ_ERR_SHAPE), q4_next 16-byte aligned (else
 *   AQ_ERR_ALIGNMENT).
 * All buffers are device memory owned by the caller; the calls enqueue on `stream` and return at once.
 * Other errors as for aq_quantize_act / aq_gemm_w4 / the chained calls. */
size_t aq_act4_bytes(int M, int K);
int aq_act4_pack(aq_handle_t h, const int8_t* q, int M, int K, void* q4, void* stream);
int aq_act4_unpack(aq_handle_t h, const void* q4, int M, int K, int8_t* q, void* stream);
int aq_quantize_act4(aq_handle_t h, const void* x_fp16, int M, int K, int scale_mode, int clip_shift_or_exp,
                     const int32_t* row_idx, void* q4, int32_t* scale_exp_out, void* workspace,
                     size_t workspace_bytes, void* stream);
int aq_gemm_w4_act4(aq_handle_t h, const void* q4, int M, int K, const void* w_packed, const void* w_scales,
                    int N, int group_size, const int32_t* scale_exp, void* y_fp16, int32_t* acc_dump,
                    void* workspace, size_t workspace_bytes, void* stream);
int aq_linear_w4a8_chain_act4(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                              const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                              const int32_t* row_idx, void* q4_next, int next_exp, int32_t* acc_dump, void* workspace,
                              size_t workspace_bytes, void* stream);
int aq_linear_w4a4_chain_act4(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                              const void* w_scales, int N, int group_size, int scale_mode, int clip_shift_or_exp,
                              const int32_t* row_idx, void* q4_next, int next_exp, int32_t* acc_dump, void* workspace,
                              size_t workspace_bytes, void* stream);

/* ---- log2 quantization of the softmax output and attention x value (paper Eq. 3, Sec. 5.1)
 * aq_log2_quantize: x_fp16 holds `count` values (any shape); max|x| is taken over all of them.
 *   k = CLIP(round(-log2(|x| / max|x|)), 0, 2^(b-1) - 1), so x ~ Sign(x) * max|x| * 2^-k. codes (int8, same
 *   shape) hold Sign(x) * (k + 1), and 0 for an exact zero (Eq. 3's Sign(0) = 0) and for NaN; +-Inf count as
 *   65504. max_bits_out (device, may be NULL) receives the fp16 bit pattern of max|x| in its low 16 bits.
 *   bits 8 or 4. The rounding is exact (decided with integers).
 * aq_attn_v_log2: P as such codes [H,M,J] (H heads, M query rows, J key rows) times V as int8 codes
 *   [H,J,D] of aq_quantize_act (with its exponent on the device):
 *     acc[h,m,d] = sum_j Sign_j * (v[h,j,d] << (kmax - k_j)),   y = fp16(max|P| * 2^(e_v - kmax) * acc).
 *   Every product is a shift. bits must be 4 (kmax = 7: with 8-bit codes the shifts would reach 127 and
 *   no integer accumulator holds them). D % 4 == 0, 256 % (D/4) == 0, D <= 1024, J <= 65536. acc_dump: NULL
 *   or int32 [H,M,D]. */
int aq_log2_quantize(aq_handle_t h, const void* x_fp16, long long count, int bits, int8_t* codes,
                     uint32_t* max_bits_out, void* workspace, size_t workspace_bytes, void* stream);
int aq_attn_v_log2(aq_handle_t h, const int8_t* p_codes, const uint32_t* p_max_bits, const int8_t* v_codes,
                   const int32_t* v_scale_exp, int H, int M, int J, int D, int bits, void* y_fp16, int32_t* acc_dump,
                   void* stream);
/* The same result on the tensor cores for a non-negative P (a softmax output), 4-bit codes: the factor
 * 2^(kmax - k) is then an unsigned byte and the sums are a u8 x s8 -> s32 contraction over j
 * (tcgen05.mma kind::i8, operands staged by TMA, accumulator in tensor memory). D is 64 or 128,
 * J % 16 == 0; y must be 16-byte aligned. The workspace (aq_attn_workspace_bytes) holds a control block
 * and the transposed value codes (the codes of P become byte factors tile by tile inside the product kernel). A negative code in P is an error: it is counted as 0
 * and aq_check_workspace on this workspace then returns AQ_ERR_INVALID_ARG. */
/* Query x key scores on int8 (or 4-bit, stored in int8) codes of aq_quantize_act, reduction over the head
 * dimension (Sec. 5.1): s[h,m,j] = fp16( 2^(e_q + e_k) * sum_d q[h,m,d] * k[h,j,d] ), q [H,M,D], k [H,J,D],
 * s [H,M,J]. D must be 128, J % 8 == 0; all three 16-byte aligned. workspace: 256 bytes (control block). */
int aq_attn_qk_tc(aq_handle_t h, const int8_t* q_codes, const int32_t* q_scale_exp, const int8_t* k_codes,
                  const int32_t* k_scale_exp, int H, int M, int J, int D, void* s_fp16, void* workspace,
                  size_t workspace_bytes, void* stream);
/* The two calls that spare the tensor-core route its conversion pass over P (Eq. 3 with 4-bit codes of a
 * non-negative input): aq_log2_quantize_factors writes, instead of the code, the byte 2^(kmax - k) =
 * 128 >> k that multiplies the value code (0 for an exact zero or NaN; a negative input is an error that
 * aq_check_workspace on this workspace reports as AQ_ERR_INVALID_ARG, its factor is 0), i.e. exactly what
 * aq_attn_v_log2_tc derives from the codes of aq_log2_quantize(bits = 4); aq_attn_v_factors_tc is
 * aq_attn_v_log2_tc on those bytes (p_factors [H,M,J], 16-byte aligned). Same results bit for bit. */
int aq_log2_quantize_factors(aq_handle_t h, const void* x_fp16, long long count, uint8_t* factors,
                             uint32_t* max_bits_out, void* workspace, size_t workspace_bytes, void* stream);
int aq_attn_v_factors_tc(aq_handle_t h, const uint8_t* p_factors, const uint32_t* p_max_bits, const int8_t* v_codes,
                         const int32_t* v_scale_exp, int H, int M, int J, int D, void* y_fp16, void* workspace,
                         size_t workspace_bytes, void* stream);
size_t aq_attn_workspace_bytes(int H, int M, int J, int D);
int aq_attn_v_log2_tc(aq_handle_t h, const int8_t* p_codes, const uint32_t* p_max_bits, const int8_t* v_codes,
                      const int32_t* v_scale_exp, int H, int M, int J, int D, void* y_fp16, void* workspace,
                      size_t workspace_bytes, void* stream);

/* ---- progressive pruning schedule (paper Eq. 9; host only, no GPU work)
 * With pruning at m layers and the ratio beta of tokens to be gone after the last of them, every
 * pruning layer drops the fraction gamma = 1 - (1 - beta)^(1/m) of what reaches it. Writes
 * n_keep_out[i], i = 0..m-1, the tokens kept after pruning layer i, starting from M tokens:
 * n_keep_out[i] = ceil(n_keep_out[i-1] * (1 - gamma)) (at least 1), and *gamma_out (may be NULL).
 * Each n_keep_out[i] is the n_keep argument of aq_token_select at that layer.
 * Returns AQ_ERR_INVALID_ARG unless M >= 1, m >= 1, 0 <= beta < 1. */
int aq_prune_schedule(int M, double beta, int m, int32_t* n_keep_out, double* gamma_out);

/* ---- host-buffer convenience (SYNCHRONIZES the stream before returning)
 * x_host fp16 [M,K] and y_host fp16 [M,N] are HOST pointers (pinned memory gives the best
 * rate). Copies x to the device scratch, runs the layer with `bits` (8 or 4), copies y
 * back. device_scratch must hold aq_linear_host_scratch_bytes() bytes. */
size_t aq_linear_host_scratch_bytes(int M, int K, int N, int group_size);
int aq_linear_host(aq_handle_t h, int bits, const void* x_host, int M, int K,
                   const void* w_packed, const void* w_scales, int N, int group_size,
                   int scale_mode, int clip_shift_or_exp, void* y_host, void* device_scratch,
                   size_t scratch_bytes, void* stream);
/* The same without the final synchronisation: the two copies and the layer are enqueued on `stream`
 * and the call returns. x_host, y_host (pinned, or the copies are not asynchronous) and device_scratch
 * belong to the call until the stream has been synchronised; y_host is valid from then on. Calls on
 * different streams, each with its own scratch, overlap their copies (one direction each) and their
 * kernels. */
int aq_linear_host_async(aq_handle_t h, int bits, const void* x_host, int M, int K,
                         const void* w_packed, const void* w_scales, int N, int group_size,
                         int scale_mode, int clip_shift_or_exp, void* y_host, void* device_scratch,
                         size_t scratch_bytes, void* stream);

/* SYNCHRONIZES the stream, then reports whether a kernel of the most recent call that used
 * this workspace gave up on a bounded wait (AQ_ERR_DEVICE_TIMEOUT); AQ_OK otherwise. Every
 * aq_linear_* / aq_gemm_w4 / aq_quantize_act call clears the record when it starts. */
int aq_check_workspace(aq_handle_t h, const void* workspace, void* stream);

/* ---- measurement aid: the tensor cores' int8 rate on this GPU (the denominator of the roofline of
 * the prefill product, Sec. 4.4's integer matrix multiplication)
 * Enqueues one kernel in which every SM issues iters x 4 tcgen05.mma kind::i8 instructions of
 * 128 x 256 x 32 on operands that stay in place (A from tensor memory when a_from_tmem != 0, as in the
 * product kernel, else from shared memory), with no loads and no epilogue. *ops_out (host, may be NULL)
 * receives the integer operations of the launch (2 per multiply-add); time the launch with events on
 * `stream`. workspace: 256 bytes (control block; aq_check_workspace reports a wait that gave up).
 * 1 <= iters <= 2^24. */
int aq_probe_int8_mma(aq_handle_t h, int iters, int a_from_tmem, double* ops_out, void* workspace,
                      size_t workspace_bytes, void* stream);

/* ---- the layer without any caller-provided or allocated scratch
 * (The paper has no counterpart to this call: it exists for the way some programs must use
 * the library, not for anything the method computes.)
 *
 * Same result as aq_linear_w4a8 with row_idx = NULL and acc_dump = NULL, but the scratch the
 * layer needs (the control block and the int8 activation codes, see aq_workspace_bytes) lives
 * in a fixed buffer inside the library instead of a workspace from the caller. It is meant for
 * callers that may not allocate device memory at the point of the call: code running inside a
 * memory pool that has already handed out the whole device, plugin and serving hosts that
 * forbid cudaMalloc after start-up because an allocation synchronizes the device and can fail
 * late, and real-time loops where an out-of-memory error must be impossible by construction.
 * This call performs no cudaMalloc / cudaFree and calls nothing that allocates.
 *
 * Limits and rules
 *  - aq_workspace_min_bytes(M, K, N, group_size) = 256 + up256(M*K) + up256(M) + up256(4*N)
 *    (up256 rounds up to a multiple of 256) must not exceed AQ_NOALLOC_SCRATCH_BYTES: M*K up to
 *    16 Mi codes as long as M + 4*N stays under 64 KiB (2048 x 8192 or 4096 x 4096 activations with
 *    N <= 15360), and any N when M*K is smaller by 4*N + M bytes. Larger sizes are refused with
 *    AQ_ERR_TOO_LARGE and nothing is enqueued; use aq_linear_w4a8 with your own workspace then.
 *    What the buffer has left beyond that minimum serves the per-group kernel's shared tiles; a
 *    shape that would want more than is left runs without sharing (see aq_workspace_min_bytes).
 *  - The buffer is a static device array: every GPU on which the library is loaded holds
 *    AQ_NOALLOC_SCRATCH_BYTES of device memory until the process exits.
 *  - The first call on each device looks up the buffer's device address (a one-time,
 *    host-side set-up that needs that device to be current). With lazy module loading (the CUDA
 *    default) that look-up is also the moment the driver loads the library's device code and
 *    reserves the buffer, so it can fail with AQ_ERR_CUDA when the device is already full. Make
 *    that first call at start-up: before a memory pool takes the rest of the device and before
 *    starting any stream capture.
 *  - All calls on a device share the one buffer, and it keeps the previous call's contents; the
 *    call itself clears the part that must start at zero. Two calls that can overlap on the
 *    GPU (different streams without ordering) race on the buffer: order them, or use
 *    aq_linear_w4a8 with separate workspaces.
 *  - The handle's device must be the current device.
 *  - aq_check_noalloc is aq_check_workspace for the built-in buffer (whose address callers do not
 *    have): it SYNCHRONIZES the stream and reports whether a kernel of the last call gave up on a
 *    bounded wait. */
#define AQ_NOALLOC_SCRATCH_BYTES ((size_t)16 * 1024 * 1024 + 65536 + 256)
int aq_linear_w4a8_noalloc(aq_handle_t h, const void* x_fp16, int M, int K, const void* w_packed,
                           const void* w_scales, int N, int group_size, int scale_mode,
                           int clip_shift_or_exp, void* y_fp16, void* stream);
int aq_check_noalloc(aq_handle_t h, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AGILEQ_H_ */

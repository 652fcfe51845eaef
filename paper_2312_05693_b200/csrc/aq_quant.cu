// Activation side: layer-wise absolute maximum, power-of-two quantization to int8 / int4
// codes (paper Eq. 1, Eq. 2 / Eq. 5 with zp = 0, layer-wise scale of Sec. 4.4), and the
// token selection / gather of Eq. 4.
#include <cooperative_groups.h>

#include "aq_common.cuh"
#include "aq_quant_math.cuh"

namespace cg = cooperative_groups;

namespace aq {

namespace {

constexpr int kQuantThreads = 256;

// The half2 route with TRIP factors (4-bit codes): lane k multiplies by 2^-(e + alpha_k), built from
// the factor byte as a half bit pattern (exponent field 15 - e - alpha_k, which must be 1..30),
// clamps to [-8, 7], rounds by adding and removing 1536, multiplies by 2^alpha_k (exact, |result|
// <= 128) and adds 1536 again so that the value's two's-complement byte sits in the low 8 bits.
__device__ __forceinline__ void quantize8_half2_trip(const uint4& d, int e, const uint2& al, uint32_t& w0, uint32_t& w1) {
    const __half2* h = reinterpret_cast<const __half2*>(&d);
    const __half2 bias = __floats2half2_rn(1536.0f, 1536.0f);
    const __half2 lo2 = __floats2half2_rn(-8.0f, -8.0f), hi2 = __floats2half2_rn(7.0f, 7.0f);
    const uint32_t inv_base = (uint32_t)(15 - e) * 0x04000400u;              // both lanes: (15 - e) << 10
    const uint32_t one_base = 15u * 0x04000400u;                            // 1.0 in both lanes
    uint32_t r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t word = i < 2 ? al.x : al.y;
        const uint32_t a0 = (word >> (16 * (i & 1))) & 0xFFu, a1 = (word >> (16 * (i & 1) + 8)) & 0xFFu;
        const uint32_t apair = (a0 | (a1 << 16)) << 10;
        uint32_t ib = inv_base - apair, sb = one_base + apair;
        __half2 t = __hmul2(h[i], *reinterpret_cast<__half2*>(&ib));
        const uint32_t ok = __heq2_mask(t, t);                              // clears NaN lanes
        uint32_t tb = *reinterpret_cast<uint32_t*>(&t) & ok;
        t = *reinterpret_cast<__half2*>(&tb);
        t = __hsub2(__hadd2(__hmin2(__hmax2(t, lo2), hi2), bias), bias);    // the 4-bit code, rounded to nearest even
        t = __hadd2(__hmul2(t, *reinterpret_cast<__half2*>(&sb)), bias);
        r[i] = *reinterpret_cast<uint32_t*>(&t);
    }
    w0 = __byte_perm(r[0], r[1], 0x6420);
    w1 = __byte_perm(r[2], r[3], 0x6420);
}

__device__ __forceinline__ uint4 quantize16_fp32(const uint4& d0, const uint4& d1, int e, float lo, float hi,
                                                 const uint4* al) {
    uint2 a0, a1;
    if (al) { a0 = make_uint2(al->x, al->y); a1 = make_uint2(al->z, al->w); }
    const uint2 r0 = quantize8_fp32(d0, e, lo, hi, al ? &a0 : nullptr);
    const uint2 r1 = quantize8_fp32(d1, e, lo, hi, al ? &a1 : nullptr);
    return make_uint4(r0.x, r0.y, r1.x, r1.y);
}

// ---- quantize: 16 halves in (two 16-byte loads), 16 codes out (one 16-byte store) -----
__global__ void __launch_bounds__(kQuantThreads)
quantize_kernel(const uint4* __restrict__ x, int M, int vec_per_row /* 16-element units */,
                const int32_t* __restrict__ row_idx, int bits, int scale_mode, int clip_shift_or_exp,
                Control* __restrict__ ctl, uint4* __restrict__ q, int32_t* __restrict__ scale_exp_out,
                const uint4* __restrict__ alpha, int k_max) {
    const int e = scale_mode == AQ_SCALE_DYNAMIC
                      ? layer_exponent_from_bits(ctl->absmax_bits, bits) - clip_shift_or_exp - k_max
                      : clip_shift_or_exp;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctl->scale_exp = e;
        if (scale_exp_out) *scale_exp_out = e;
    }
    const float lo = -(float)(1 << (bits - 1)), hi = (float)((1 << (bits - 1)) - 1);
    const size_t total = (size_t)M * vec_per_row;
    const size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= total) return;
    const int m = (int)(v / vec_per_row), c = (int)(v % vec_per_row);
    const size_t src = ((size_t)(row_idx ? row_idx[m] : m) * vec_per_row + c) * 2;
    const uint4 d0 = __ldg(x + src), d1 = __ldg(x + src + 1);
    uint4 al;
    if (alpha) al = __ldg(alpha + c);
    q[v] = quantize16_fp32(d0, d1, e, lo, hi, alpha ? &al : nullptr);
}

// ---- small activations (decode): maximum, exponent and codes in ONE kernel -------------
// One cluster of 8 CTAs x 512 threads holds the whole activation in registers (up to 8 vectors of
// 8 halves per thread), so x is read once; the CTAs' maxima are exchanged through distributed
// shared memory. The kernel also initialises the control block, so no memset precedes it.
constexpr int kSmallCtas = 8, kSmallThreads = 512, kSmallVecs = 8;
constexpr size_t kSmallMaxElems = (size_t)kSmallCtas * kSmallThreads * kSmallVecs * 8;   // 262144

__global__ void __cluster_dims__(kSmallCtas, 1, 1) __launch_bounds__(kSmallThreads)
quantize_small_kernel(const uint4* __restrict__ x, int M, int vec_per_row, const int32_t* __restrict__ row_idx,
                      int bits, int scale_mode, int clip_shift_or_exp, Control* __restrict__ ctl,
                      uint2* __restrict__ q, int32_t* __restrict__ scale_exp_out, const uint2* __restrict__ alpha,
                      int k_max, int early_dependents) {
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ unsigned int warp_max[kSmallThreads / 32];
    __shared__ unsigned int slots[kSmallCtas];
    // The launch allows programmatic stream serialization, so this grid may be set up while the kernel
    // ahead of it drains; nothing is read or written before that kernel has completed. Only then is the
    // dependent launch allowed: a product kernel launched the same way behind this one may be set up on
    // the idle SMs and fetch its weights while this one runs (it waits for this grid before it reads the
    // codes), and by then everything that preceded this kernel on the stream is complete.
    // early_dependents: the caller has promised that nothing in flight writes the weights the product kernel
    // fetches ahead of its own wait, so that kernel may be set up before this one's wait ends as well.
    if (early_dependents) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!early_dependents) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int rank = (int)cluster.block_rank();
    const int total = M * vec_per_row;
    uint4 buf[kSmallVecs];
    __half2 m2 = __float2half2_rn(0.0f);
    // all loads first, then the maximum: the loads of a thread are in flight together (one memory round
    // trip for the whole activation instead of one per vector)
#pragma unroll
    for (int i = 0; i < kSmallVecs; ++i) {
        const int v = (i * kSmallCtas + rank) * kSmallThreads + (int)threadIdx.x;
        buf[i] = make_uint4(0, 0, 0, 0);
        if (v < total) {
            const int m = v / vec_per_row, c = v % vec_per_row;
            buf[i] = __ldg(x + (size_t)(row_idx ? row_idx[m] : m) * vec_per_row + c);
        }
    }
#pragma unroll
    for (int i = 0; i < kSmallVecs; ++i) {
        const __half2* h = reinterpret_cast<const __half2*>(&buf[i]);
#pragma unroll
        for (int k = 0; k < 4; ++k) m2 = __hmax2(m2, __habs2(h[k]));   // NaN operands are dropped; absent vectors are zero
    }
    unsigned int bits_max = max((unsigned int)__half_as_ushort(__low2half(m2)),
                                (unsigned int)__half_as_ushort(__high2half(m2)));
    if (bits_max > 0x7C00u) bits_max = 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bits_max = max(bits_max, __shfl_xor_sync(0xFFFFFFFFu, bits_max, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = bits_max;
    __syncthreads();
    if (threadIdx.x < kSmallCtas) {
        unsigned int b = 0;
        for (int w = 0; w < kSmallThreads / 32; ++w) b = max(b, warp_max[w]);
        *cluster.map_shared_rank(&slots[rank], (int)threadIdx.x) = b;   // my maximum into every CTA's table
    }
    cluster.sync();
    unsigned int all = 0;
#pragma unroll
    for (int r = 0; r < kSmallCtas; ++r) all = max(all, slots[r]);
    const int e = scale_mode == AQ_SCALE_DYNAMIC ? layer_exponent_from_bits(all, bits) - clip_shift_or_exp - k_max
                                                 : clip_shift_or_exp;
    if (rank == 0 && threadIdx.x == 0) {
        ctl->absmax_bits = all;
        ctl->scale_exp = e;
        ctl->status = 0;
        ctl->counter = 0;
        if (scale_exp_out) *scale_exp_out = e;
    }
    if (rank == 0 && threadIdx.x < 57) ctl->split_flags[threadIdx.x] = 0;    // the product kernel's shared-tile bits
    const float lo = -(float)(1 << (bits - 1)), hi = (float)((1 << (bits - 1)) - 1);
    if (alpha == nullptr && e >= -14 && e <= 14) {           // 2^-e is a normal half: codes in half2 arithmetic
        const __half2 inv2 = __float2half2_rn(__int_as_float((127 - e) << 23));
        const __half2 lo2 = __float2half2_rn(lo), hi2 = __float2half2_rn(hi);
#pragma unroll
        for (int i = 0; i < kSmallVecs; ++i) {
            const int v = (i * kSmallCtas + rank) * kSmallThreads + (int)threadIdx.x;
            if (v < total) {
                uint2 w;
                quantize8_half2(buf[i], inv2, lo2, hi2, w.x, w.y);
                q[v] = w;
            }
        }
        return;
    }
#pragma unroll
    for (int i = 0; i < kSmallVecs; ++i) {
        const int v = (i * kSmallCtas + rank) * kSmallThreads + (int)threadIdx.x;
        if (v < total) {
            uint2 al;
            if (alpha) al = __ldg(alpha + v % vec_per_row);
            q[v] = quantize8_fp32(buf[i], e, lo, hi, alpha ? &al : nullptr);
        }
    }
}

// ---- larger activations, dynamic scale: maximum, exponent and codes in ONE cooperative kernel ----
// One CTA per SM takes a contiguous share of X. First pass: 16-byte loads from HBM, running maximum,
// and the loaded vectors are parked in shared memory (as much of the share as fits). The CTAs then
// meet at a counter in the control block (all are resident: the launch is cooperative; the wait is
// bounded all the same), every CTA derives the exponent from the global maximum, and the second
// pass quantizes from shared memory (from L2 for what did not fit), so X crosses HBM once.
constexpr int kFusedThreads = 1024;
constexpr unsigned int kFusedWaitCode = 10;            // status value when the meeting point times out
constexpr unsigned long long kFusedWaitCycles = 2000000000ull;   // ~1 s

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void __launch_bounds__(kFusedThreads, 1)
quantize_fused_kernel(const uint4* __restrict__ x, int M, int units_per_row /* 16-element units */,
                      const int32_t* __restrict__ row_idx, int bits, int clip_shift, Control* __restrict__ ctl,
                      uint4* __restrict__ q, int32_t* __restrict__ scale_exp_out, unsigned int cache_units,
                      unsigned int units_per_cta, const uint4* __restrict__ alpha, int k_max) {
    extern __shared__ uint4 fused_cache[];             // [2][cache_units]: first and second vector of a unit
    __shared__ unsigned int warp_max[kFusedThreads / 32];
    __shared__ int e_shared;
    __shared__ int gave_up;
    const size_t total = (size_t)M * units_per_row;
    const size_t u0 = (size_t)blockIdx.x * units_per_cta;
    const size_t u1 = u0 + units_per_cta < total ? u0 + units_per_cta : total;
    // a product kernel launched with programmatic stream serialization may be scheduled as soon as this
    // grid's CTAs leave their SMs (it waits for this grid before it reads the codes); no effect otherwise
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    __half2 m2 = __float2half2_rn(0.0f);
    // four units (eight 16-byte loads) in flight per thread before the first is used: a CTA's share is a few
    // units per thread, so the pass is one or two memory round trips rather than one per unit
    constexpr int kInFlight = 4;
    for (size_t ub = u0 + threadIdx.x; ub < u1; ub += (size_t)kFusedThreads * kInFlight) {
        uint4 d0[kInFlight], d1[kInFlight];
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) {
            const size_t u = ub + (size_t)i * kFusedThreads;
            if (u < u1) {
                const int m = (int)(u / units_per_row), c = (int)(u % units_per_row);
                const size_t src = ((size_t)(row_idx ? row_idx[m] : m) * units_per_row + c) * 2;
                d0[i] = __ldg(x + src); d1[i] = __ldg(x + src + 1);
            } else {
                d0[i] = make_uint4(0u, 0u, 0u, 0u); d1[i] = d0[i];
            }
        }
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) {
            const size_t u = ub + (size_t)i * kFusedThreads;
            if (u < u1) {
                const unsigned int local = (unsigned int)(u - u0);
                if (local < cache_units) { fused_cache[local] = d0[i]; fused_cache[cache_units + local] = d1[i]; }
            }
            const __half2* h0 = reinterpret_cast<const __half2*>(&d0[i]);
            const __half2* h1 = reinterpret_cast<const __half2*>(&d1[i]);
#pragma unroll
            for (int k = 0; k < 4; ++k) m2 = __hmax2(m2, __hmax2(__habs2(h0[k]), __habs2(h1[k])));   // NaN operands are dropped
        }
    }
    unsigned int bmax = max((unsigned int)__half_as_ushort(__low2half(m2)),
                            (unsigned int)__half_as_ushort(__high2half(m2)));
    if (bmax > 0x7C00u) bmax = 0;                                       // never publish NaN
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) bmax = max(bmax, __shfl_xor_sync(0xFFFFFFFFu, bmax, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = bmax;
    __syncthreads();
    if (threadIdx.x < 32) {
        unsigned int b = warp_max[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xFFFFFFFFu, b, o));
        if (threadIdx.x == 0) {
            if (b != 0) atomicMax(&ctl->absmax_bits, b);
            __threadfence();
            atomicAdd(&ctl->counter, 1u);
            // meeting point: every CTA has added its maximum once the counter reaches the grid size
            const long long t0 = clock64();
            int failed = 0;
            while (ld_acquire_u32(&ctl->counter) < gridDim.x) {
                if ((unsigned long long)(clock64() - t0) > kFusedWaitCycles) { failed = 1; break; }
                __nanosleep(100);
            }
            gave_up = failed;
            e_shared = layer_exponent_from_bits(ld_acquire_u32(&ctl->absmax_bits), bits) - clip_shift - k_max;
        }
    }
    __syncthreads();
    if (gave_up) {
        if (threadIdx.x == 0) atomicCAS(&ctl->status, 0u, kFusedWaitCode);
        return;
    }
    const int e = e_shared;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctl->scale_exp = e;
        if (scale_exp_out) *scale_exp_out = e;
    }
    const float inv = __int_as_float((127 - e) << 23);      // 2^-e, |e| <= 40
    const float lo = -(float)(1 << (bits - 1)), hi = (float)((1 << (bits - 1)) - 1);
    const bool fast = alpha == nullptr && e >= -14 && e <= 14;   // 2^-e is a normal half
    const bool fast_trip = alpha != nullptr && bits == 4 && e >= -14 && e <= 10;   // so is 2^-(e + alpha), alpha <= 4
    const __half2 inv2 = __float2half2_rn(fast ? inv : 1.0f), lo2 = __float2half2_rn(lo), hi2 = __float2half2_rn(hi);
#pragma unroll 2
    for (size_t u = u0 + threadIdx.x; u < u1; u += kFusedThreads) {
        const unsigned int local = (unsigned int)(u - u0);
        uint4 d0, d1;
        if (local < cache_units) {
            d0 = fused_cache[local]; d1 = fused_cache[cache_units + local];      // this thread's own stores
        } else {
            const int m = (int)(u / units_per_row), c = (int)(u % units_per_row);
            const size_t src = ((size_t)(row_idx ? row_idx[m] : m) * units_per_row + c) * 2;
            d0 = __ldg(x + src); d1 = __ldg(x + src + 1);
        }
        uint32_t out[4];
        if (fast) {
            quantize8_half2(d0, inv2, lo2, hi2, out[0], out[1]);
            quantize8_half2(d1, inv2, lo2, hi2, out[2], out[3]);
            q[u] = make_uint4(out[0], out[1], out[2], out[3]);
        } else if (fast_trip) {
            const uint4 al = __ldg(alpha + (size_t)(u % units_per_row));
            quantize8_half2_trip(d0, e, make_uint2(al.x, al.y), out[0], out[1]);
            quantize8_half2_trip(d1, e, make_uint2(al.z, al.w), out[2], out[3]);
            q[u] = make_uint4(out[0], out[1], out[2], out[3]);
        } else {
            uint4 al;
            if (alpha) al = __ldg(alpha + (size_t)(u % units_per_row));
            q[u] = quantize16_fp32(d0, d1, e, lo, hi, alpha ? &al : nullptr);
        }
    }
}

// ---- zero-point variant (Eq. 2, Eq. 5-7 with alpha = 0, power-of-two scale) ---------------
// Order-preserving map of a float's bits to an unsigned integer, so that atomicMin / atomicMax
// on the keys give the minimum / maximum value.
__device__ __forceinline__ unsigned int float_key(float f) {
    const unsigned int b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned int k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}
constexpr unsigned int kZeroKey = 0x80000000u;         // key of +0.0: the range always contains 0

// 8 halves -> 8 stored codes (q - 2^(b-1)) of the zero-point quantizer in half2 arithmetic, for
// exponents whose 2^-e is a normal half. The product by 2^-e is exact (or saturates and is clamped);
// NaN lanes are cleared to 0, which becomes the code zp; clamping rint(t) + zp to [0, qr] equals
// clamping t to [-zp, qr - zp] before rounding (integer bounds); adding 1536 rounds to nearest even;
// adding the integer zp - 2^(b-1) keeps the sum inside [1024, 2048), so the code's byte is the low
// 8 bits of the half's bit pattern.
__device__ __forceinline__ void quantize8_half2_asym(const uint4& d, __half2 inv2, __half2 lo2, __half2 hi2,
                                                     __half2 shift2, uint32_t& w0, uint32_t& w1) {
    const __half2* h = reinterpret_cast<const __half2*>(&d);
    const __half2 bias = __floats2half2_rn(1536.0f, 1536.0f);
    uint32_t r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __half2 t = __hmul2(h[i], inv2);
        const uint32_t ok = __heq2_mask(t, t);
        uint32_t tb = *reinterpret_cast<uint32_t*>(&t) & ok;
        t = *reinterpret_cast<__half2*>(&tb);
        t = __hadd2(__hadd2(__hmin2(__hmax2(t, lo2), hi2), bias), shift2);
        r[i] = *reinterpret_cast<uint32_t*>(&t);
    }
    w0 = __byte_perm(r[0], r[1], 0x6420);
    w1 = __byte_perm(r[2], r[3], 0x6420);
}

// One cooperative kernel, as quantize_fused_kernel: first pass minimum and maximum (16-byte loads, the
// share parked in shared memory), meeting point, e and zp in binary64 by one thread per CTA, second
// pass codes from shared memory.
__global__ void __launch_bounds__(kFusedThreads, 1)
quantize_asym_fused_kernel(const uint4* __restrict__ x, int M, int units_per_row /* 16-element units */,
                           const int32_t* __restrict__ row_idx, int bits, Control* __restrict__ ctl,
                           uint4* __restrict__ q, int32_t* __restrict__ scale_exp_out,
                           int32_t* __restrict__ zero_point_out, unsigned int cache_units, unsigned int units_per_cta) {
    extern __shared__ uint4 fused_cache[];             // [2][cache_units]
    __shared__ unsigned int warp_min[kFusedThreads / 32], warp_maxk[kFusedThreads / 32];
    __shared__ int params[3];                          // e, zp, gave up
    const size_t total = (size_t)M * units_per_row;
    const size_t u0 = (size_t)blockIdx.x * units_per_cta;
    const size_t u1 = u0 + units_per_cta < total ? u0 + units_per_cta : total;

    __half2 lo2 = __float2half2_rn(0.0f), hi2 = __float2half2_rn(0.0f);      // the range always contains 0
#pragma unroll 2
    for (size_t u = u0 + threadIdx.x; u < u1; u += kFusedThreads) {
        const int m = (int)(u / units_per_row), c = (int)(u % units_per_row);
        const size_t src = ((size_t)(row_idx ? row_idx[m] : m) * units_per_row + c) * 2;
        const uint4 d0 = __ldg(x + src), d1 = __ldg(x + src + 1);
        const unsigned int local = (unsigned int)(u - u0);
        if (local < cache_units) { fused_cache[local] = d0; fused_cache[cache_units + local] = d1; }
        const __half2* h0 = reinterpret_cast<const __half2*>(&d0);
        const __half2* h1 = reinterpret_cast<const __half2*>(&d1);
#pragma unroll
        for (int i = 0; i < 4; ++i) {                                        // NaN operands are dropped
            lo2 = __hmin2(lo2, __hmin2(h0[i], h1[i]));
            hi2 = __hmax2(hi2, __hmax2(h0[i], h1[i]));
        }
    }
    // +-Inf count as the largest half
    const float lo = fmaxf(fminf(__low2float(lo2), __high2float(lo2)), -65504.0f);
    const float hi = fminf(fmaxf(__low2float(hi2), __high2float(hi2)), 65504.0f);
    unsigned int kmin = float_key(lo), kmax = float_key(hi);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, o));
    }
    if ((threadIdx.x & 31) == 0) { warp_min[threadIdx.x >> 5] = kmin; warp_maxk[threadIdx.x >> 5] = kmax; }
    __syncthreads();
    if (threadIdx.x < 32) {
        kmin = warp_min[threadIdx.x];
        kmax = warp_maxk[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, o));
            kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, o));
        }
        if (threadIdx.x == 0) {
            // the control block is cleared to 0: keys are stored relative to the key of 0.0
            if (kmax > kZeroKey) atomicMax(&ctl->max_key, kmax - kZeroKey);
            if (kmin < kZeroKey) atomicMax(&ctl->min_key, kZeroKey - kmin);
            __threadfence();
            atomicAdd(&ctl->counter, 1u);
            const long long t0 = clock64();
            int failed = 0;
            while (ld_acquire_u32(&ctl->counter) < gridDim.x) {
                if ((unsigned long long)(clock64() - t0) > kFusedWaitCycles) { failed = 1; break; }
                __nanosleep(100);
            }
            const double qr = (double)((1 << bits) - 1);
            const double dhi = (double)key_float(kZeroKey + ld_acquire_u32(&ctl->max_key));
            const double dlo = (double)key_float(kZeroKey - ld_acquire_u32(&ctl->min_key));
            const double range = dhi - dlo;
            int ee = 0;
            if (range > 0.0) {
                int ex;
                frexp(range / qr, &ex);              // a first guess within one of the answer
                ee = ex;
                while (ldexp(qr, ee) < range) ++ee;
                while (ldexp(qr, ee - 1) >= range) --ee;
            }
            params[0] = ee;
            params[1] = (int)fmin(fmax(rint(ldexp(-dlo, -ee)), 0.0), qr);
            params[2] = failed;
        }
    }
    __syncthreads();
    if (params[2]) {
        if (threadIdx.x == 0) atomicCAS(&ctl->status, 0u, kFusedWaitCode);
        return;
    }
    const int e = params[0], zp = params[1];
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctl->scale_exp = e;
        ctl->zero_point = zp;
        if (scale_exp_out) *scale_exp_out = e;
        if (zero_point_out) *zero_point_out = zp;
    }
    const int qr_i = (1 << bits) - 1, half_range = 1 << (bits - 1);
    const float inv = __int_as_float((127 - e) << 23);      // 2^-e
    const float fzp = (float)zp, fqr = (float)qr_i;
    const bool fast = e >= -14 && e <= 14;                   // 2^-e is a normal half
    const __half2 inv2 = __float2half2_rn(fast ? inv : 1.0f);
    const __half2 clo2 = __float2half2_rn(-fzp), chi2 = __float2half2_rn(fqr - fzp);
    const __half2 shift2 = __float2half2_rn((float)(zp - half_range));
#pragma unroll 2
    for (size_t u = u0 + threadIdx.x; u < u1; u += kFusedThreads) {
        const unsigned int local = (unsigned int)(u - u0);
        uint4 d0, d1;
        if (local < cache_units) {
            d0 = fused_cache[local]; d1 = fused_cache[cache_units + local];      // this thread's own stores
        } else {
            const int m = (int)(u / units_per_row), c = (int)(u % units_per_row);
            const size_t src = ((size_t)(row_idx ? row_idx[m] : m) * units_per_row + c) * 2;
            d0 = __ldg(x + src); d1 = __ldg(x + src + 1);
        }
        uint32_t out[4];
        if (fast) {
            quantize8_half2_asym(d0, inv2, clo2, chi2, shift2, out[0], out[1]);
            quantize8_half2_asym(d1, inv2, clo2, chi2, shift2, out[2], out[3]);
        } else {
            const __half* h0 = reinterpret_cast<const __half*>(&d0);
            const __half* h1 = reinterpret_cast<const __half*>(&d1);
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                uint32_t word = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int i = 4 * w + b;
                    const float t = __half2float(i < 8 ? h0[i] : h1[i - 8]) * inv;    // exact
                    int code = zp;                                                    // NaN: value 0
                    if (t == t) code = (int)fminf(fmaxf(rintf(t) + fzp, 0.0f), fqr);
                    word |= ((uint32_t)(code - half_range) & 0xFFu) << (8 * b);
                }
                out[w] = word;
            }
        }
        q[u] = make_uint4(out[0], out[1], out[2], out[3]);
    }
}

__global__ void chan_offsets_kernel(const float* __restrict__ r, int N, int bits, const Control* __restrict__ ctl,
                                    float* __restrict__ off) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n < N) off[n] = -(float)(ctl->zero_point - (1 << (bits - 1))) * r[n];
}

// ---- TRIP calibration (Eq. 8 with the clipping of Eq. 5) ---------------------------------
__global__ void __launch_bounds__(256)
absmax_plain_kernel(const __half* __restrict__ x, int M, int K, const int32_t* __restrict__ row_idx,
                    Control* __restrict__ ctl) {
    const size_t total = (size_t)M * K;
    unsigned int b = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / K), k = (int)(i % K);
        const unsigned int hb = __half_as_ushort(x[(size_t)(row_idx ? row_idx[m] : m) * K + k]) & 0x7FFFu;
        if (hb <= 0x7C00u) b = max(b, hb);                                  // NaN is ignored
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xFFFFFFFFu, b, o));
    if ((threadIdx.x & 31) == 0 && b != 0) atomicMax(&ctl->absmax_bits, b);
}

// One thread per channel walks the tokens in ascending order and keeps one binary64 error sum per
// candidate factor (product and sum rounded separately), then takes the smallest factor among the
// least errors. Consecutive threads read consecutive halves of a row.
__global__ void __launch_bounds__(128)
trip_calibrate_kernel(const __half* __restrict__ x, int M, int K, const int32_t* __restrict__ row_idx, int bits,
                      int k_max, Control* __restrict__ ctl, uint8_t* __restrict__ alpha_out,
                      int32_t* __restrict__ scale_exp_out) {
    const int e = layer_exponent_from_bits(ctl->absmax_bits, bits) - k_max;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        ctl->scale_exp = e;
        if (scale_exp_out) *scale_exp_out = e;
    }
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const double lo = -(double)(1 << (bits - 1)), hi = (double)((1 << (bits - 1)) - 1);
    double err[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
    for (int m = 0; m < M; ++m) {
        const float xf = __half2float(x[(size_t)(row_idx ? row_idx[m] : m) * K + k]);
        if (!isfinite(xf)) continue;
        const double xv = (double)xf;
#pragma unroll
        for (int a = 0; a < 5; ++a) {
            if (a <= k_max) {
                const double inv = __longlong_as_double((long long)(1023 - e - a) << 52);    // 2^-(e+a)
                const double step = __longlong_as_double((long long)(1023 + e + a) << 52);   // 2^(e+a)
                const double qv = fmin(fmax(rint(__dmul_rn(xv, inv)), lo), hi);
                const double d = __dsub_rn(xv, __dmul_rn(qv, step));
                err[a] = __dadd_rn(err[a], __dmul_rn(d, d));
            }
        }
    }
    int best = 0;
    double best_err = err[0];
#pragma unroll
    for (int a = 1; a < 5; ++a)
        if (a <= k_max && err[a] < best_err) { best = a; best_err = err[a]; }
    alpha_out[k] = (uint8_t)best;
}

// ---- token selection: the n_keep highest scores, equal scores toward the lower index, ascending indices out ----
// One CTA. Scores become 32-bit keys whose unsigned order is the scores' order (-0 and +0 share a key, so
// they tie as they do in a float comparison). The key T of the n_keep-th highest score is built from the top,
// two bits per pass: a digit is the largest one for which at least n_keep keys are >= the candidate (16
// counting passes, one block-wide sum of three counts each). Every key above T is kept, and of the keys equal to T the first
// n_keep - #{key > T} in index order; one block scan over (greater, equal) counts gives each kept token its
// place in the output. Exactly n_keep indices are written whatever the scores hold (NaNs order by their bit
// patterns: positive ones above +inf, negative ones below -inf).
// REGS: M <= 4 * kSelThreads and each thread keeps its four consecutive tokens' keys in registers for all
// passes (a counting pass is then twelve compares, two rounds of warp reductions and one barrier).
constexpr int kSelThreads = 1024;
constexpr int kSelStage = 8192;           // keys held in shared memory up to this M; beyond it every pass reads the scores

__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <bool REGS>
__global__ void __launch_bounds__(kSelThreads)
token_select_kernel(const float* __restrict__ scores, int M, int n_keep, int32_t* __restrict__ idx) {
    __shared__ uint32_t skeys[REGS ? 1 : kSelStage];
    __shared__ int wsum[2][3][32];
    __shared__ unsigned long long wscan[32];
    __shared__ unsigned long long running;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const bool staged = !REGS && M <= kSelStage;
    uint32_t kreg[4] = {0u, 0u, 0u, 0u};                 // key 0 is below every candidate of the passes
    if (REGS) {
#pragma unroll
        for (int b = 0; b < 4; ++b)
            if (4 * tid + b < M) kreg[b] = score_key(__ldg(scores + 4 * tid + b));
    } else if (staged) {
        for (int j = tid; j < M; j += kSelThreads) skeys[j] = score_key(__ldg(scores + j));
    }
    if (tid == 0) running = 0ull;
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return staged ? skeys[j] : score_key(__ldg(scores + j)); };
    // One pass settles two bits of T: the counts of keys >= T | (v << shift) for v = 1, 2, 3, the same values
    // in every thread; T takes the largest v whose count still reaches n_keep. buf alternates so that a pass
    // never overwrites sums a slower warp is still reading.
    uint32_t T = 0u;
    int above = 0;            // #{ key >= T + (1 << settled digits' lowest bit) }: 0 while nothing is settled
    for (int shift = 30; shift >= 0; shift -= 2) {
        const uint32_t c1 = T | (1u << shift), c2 = T | (2u << shift), c3 = T | (3u << shift);
        int n1 = 0, n2 = 0, n3 = 0;
        if (REGS) {
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                n1 += (int)(kreg[b] >= c1); n2 += (int)(kreg[b] >= c2); n3 += (int)(kreg[b] >= c3);
            }
        } else {
            for (int j = tid; j < M; j += kSelThreads) {
                const uint32_t k = key_at(j);
                n1 += (int)(k >= c1); n2 += (int)(k >= c2); n3 += (int)(k >= c3);
            }
        }
        n1 = __reduce_add_sync(0xFFFFFFFFu, n1);
        n2 = __reduce_add_sync(0xFFFFFFFFu, n2);
        n3 = __reduce_add_sync(0xFFFFFFFFu, n3);
        const int buf = (shift >> 1) & 1;
        if (lane == 0) { wsum[buf][0][wid] = n1; wsum[buf][1][wid] = n2; wsum[buf][2][wid] = n3; }
        __syncthreads();
        n1 = __reduce_add_sync(0xFFFFFFFFu, wsum[buf][0][lane]);
        n2 = __reduce_add_sync(0xFFFFFFFFu, wsum[buf][1][lane]);
        n3 = __reduce_add_sync(0xFFFFFFFFu, wsum[buf][2][lane]);
        // counts fall with v. The candidate one digit step above the chosen one is the next v, or, for
        // v = 3, the previous pass's upper neighbour, whose count `above` already holds.
        if (n3 >= n_keep)      { T = c3; }
        else if (n2 >= n_keep) { T = c2; above = n3; }
        else if (n1 >= n_keep) { T = c1; above = n2; }
        else                   { above = n1; }
    }
    const int greater = above;                          // after the last pass the step is 1: #{ key > T }
    const int need = n_keep - greater;                  // ties at T to keep, lowest indices first

    // four consecutive tokens per thread; counts packed as (equal << 32) | greater
    for (int base = 0; base < M; base += 4 * kSelThreads) {
        const int j0 = base + 4 * tid;
        uint32_t gt = 0u, eq = 0u;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if (j0 + b < M) {
                const uint32_t k = REGS ? kreg[b] : key_at(j0 + b);
                gt |= (uint32_t)(k > T) << b;
                eq |= (uint32_t)(k == T) << b;
            }
        }
        const unsigned long long own = ((unsigned long long)__popc(eq) << 32) | (unsigned long long)__popc(gt);
        unsigned long long incl = own;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) wscan[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            unsigned long long ws = wscan[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, ws, o);
                if (lane >= o) ws += t;
            }
            wscan[lane] = ws;   // inclusive over warps
        }
        __syncthreads();
        const unsigned long long before = running + (wid ? wscan[wid - 1] : 0ull) + incl - own;
        int gt_before = (int)(uint32_t)before, eq_before = (int)(before >> 32);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            if ((gt >> b) & 1u) {
                idx[gt_before + min(eq_before, need)] = j0 + b;
                ++gt_before;
            } else if ((eq >> b) & 1u) {
                if (eq_before < need) idx[gt_before + eq_before] = j0 + b;
                ++eq_before;
            }
        }
        __syncthreads();
        if (tid == 0) running += wscan[31];
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ x, int vec_per_row, const int32_t* __restrict__ idx,
                   int n_keep, uint4* __restrict__ out) {
    const size_t total = (size_t)n_keep * vec_per_row;
    for (size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x; v < total;
         v += (size_t)gridDim.x * blockDim.x) {
        const int m = (int)(v / vec_per_row), c = (int)(v % vec_per_row);
        out[v] = __ldg(x + (size_t)idx[m] * vec_per_row + c);
    }
}

}  // namespace

cudaError_t launch_quantize(const __half* x, int M, int K, const int32_t* row_idx, int bits,
                            int scale_mode, int clip_shift_or_exp, Control* ctl, int8_t* q,
                            int32_t* scale_exp_out, const DeviceInfo& dev, cudaStream_t stream,
                            const uint8_t* alpha, int k_max) {
    (void)dev;
    const int vec_per_row = K / 16;
    const size_t total = (size_t)M * vec_per_row;
    const size_t blocks = (total + kQuantThreads - 1) / kQuantThreads;
    quantize_kernel<<<(unsigned int)blocks, kQuantThreads, 0, stream>>>(
        reinterpret_cast<const uint4*>(x), M, vec_per_row, row_idx, bits, scale_mode, clip_shift_or_exp,
        ctl, reinterpret_cast<uint4*>(q), scale_exp_out, reinterpret_cast<const uint4*>(alpha), k_max);
    return cudaGetLastError();
}

cudaError_t launch_quantize_fused(const __half* x, int M, int K, const int32_t* row_idx, int bits, int clip_shift,
                                  Control* ctl, int8_t* q, int32_t* scale_exp_out, const DeviceInfo& dev,
                                  cudaStream_t stream, const uint8_t* alpha, int k_max) {
    int units_per_row = K / 16;
    const size_t total = (size_t)M * units_per_row;
    size_t grid = (total + kFusedThreads - 1) / kFusedThreads;
    if (grid > (size_t)dev.sm_count) grid = (size_t)dev.sm_count;
    unsigned int units_per_cta = (unsigned int)((total + grid - 1) / grid);
    // shared-memory cache: the CTA's whole share when it fits, else as much as one CTA may hold
    const size_t reserve = 8192;                       // static shared memory and alignment slack
    const size_t max_cache = dev.smem_optin > reserve ? (dev.smem_optin - reserve) / 32 : 0;
    unsigned int cache_units = units_per_cta < max_cache ? units_per_cta : (unsigned int)max_cache;
    const size_t smem_bytes = (size_t)cache_units * 32;
    static SmemOptIn opt_in;            // always the device's whole opt-in size: any later share fits
    if (const cudaError_t e = opt_in.ensure(quantize_fused_kernel, dev.device, dev.smem_optin - reserve); e != cudaSuccess)
        return e;
    const uint4* xp = reinterpret_cast<const uint4*>(x);
    uint4* qp = reinterpret_cast<uint4*>(q);
    const uint4* ap = reinterpret_cast<const uint4*>(alpha);
    void* args[] = {&xp, &M, &units_per_row, &row_idx, &bits, &clip_shift, &ctl, &qp, &scale_exp_out, &cache_units,
                    &units_per_cta, &ap, &k_max};
    // cooperative: the launch fails rather than start a grid whose CTAs could not all be resident
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(quantize_fused_kernel), dim3((unsigned int)grid),
                                       dim3(kFusedThreads), args, smem_bytes, stream);
}

cudaError_t launch_trip_calibrate(const __half* x, int M, int K, const int32_t* row_idx, int bits, int k_max,
                                  Control* ctl, uint8_t* alpha_out, int32_t* scale_exp_out, const DeviceInfo& dev,
                                  cudaStream_t stream) {
    const size_t total = (size_t)M * K;
    size_t blocks = (total + 255) / 256;
    const size_t cap = (size_t)dev.sm_count * 8;
    if (blocks > cap) blocks = cap;
    absmax_plain_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(x, M, K, row_idx, ctl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    trip_calibrate_kernel<<<(K + 127) / 128, 128, 0, stream>>>(x, M, K, row_idx, bits, k_max, ctl, alpha_out,
                                                               scale_exp_out);
    return cudaGetLastError();
}

cudaError_t launch_quantize_asym(const __half* x, int M, int K, const int32_t* row_idx, int bits, Control* ctl,
                                 int8_t* q, int32_t* scale_exp_out, int32_t* zero_point_out, const DeviceInfo& dev,
                                 cudaStream_t stream) {
    int units_per_row = K / 16;
    const size_t total = (size_t)M * units_per_row;
    size_t grid = (total + kFusedThreads - 1) / kFusedThreads;
    if (grid > (size_t)dev.sm_count) grid = (size_t)dev.sm_count;
    unsigned int units_per_cta = (unsigned int)((total + grid - 1) / grid);
    const size_t reserve = 8192;
    const size_t max_cache = dev.smem_optin > reserve ? (dev.smem_optin - reserve) / 32 : 0;
    unsigned int cache_units = units_per_cta < max_cache ? units_per_cta : (unsigned int)max_cache;
    const size_t smem_bytes = (size_t)cache_units * 32;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(quantize_asym_fused_kernel, dev.device, dev.smem_optin - reserve);
        e != cudaSuccess)
        return e;
    const uint4* xp = reinterpret_cast<const uint4*>(x);
    uint4* qp = reinterpret_cast<uint4*>(q);
    void* args[] = {&xp, &M, &units_per_row, &row_idx, &bits, &ctl, &qp, &scale_exp_out, &zero_point_out, &cache_units,
                    &units_per_cta};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(quantize_asym_fused_kernel),
                                       dim3((unsigned int)grid), dim3(kFusedThreads), args, smem_bytes, stream);
}

cudaError_t launch_chan_offsets(const float* r, int N, int bits, const Control* ctl, float* off, cudaStream_t stream) {
    chan_offsets_kernel<<<(N + 255) / 256, 256, 0, stream>>>(r, N, bits, ctl, off);
    return cudaGetLastError();
}

bool quantize_small_fits(int M, int K) { return (size_t)M * (size_t)K <= kSmallMaxElems; }

cudaError_t launch_quantize_small(const __half* x, int M, int K, const int32_t* row_idx, int bits, int scale_mode,
                                  int clip_shift_or_exp, Control* ctl, int8_t* q, int32_t* scale_exp_out,
                                  cudaStream_t stream, const uint8_t* alpha, int k_max, bool early_dependents) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kSmallCtas);
    cfg.blockDim = dim3(kSmallThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;       // the kernel touches no memory before the kernel ahead of it has completed
    return cudaLaunchKernelEx(&cfg, quantize_small_kernel, reinterpret_cast<const uint4*>(x), M, K / 8, row_idx, bits,
                              scale_mode, clip_shift_or_exp, ctl, reinterpret_cast<uint2*>(q), scale_exp_out,
                              reinterpret_cast<const uint2*>(alpha), k_max, early_dependents ? 1 : 0);
}

cudaError_t launch_token_select(const float* scores, int M, int n_keep, int32_t* idx, void* scratch,
                                cudaStream_t stream) {
    (void)scratch;
    if (n_keep == 0) return cudaSuccess;
    if (M <= 4 * kSelThreads)
        token_select_kernel<true><<<1, kSelThreads, 0, stream>>>(scores, M, n_keep, idx);
    else
        token_select_kernel<false><<<1, kSelThreads, 0, stream>>>(scores, M, n_keep, idx);
    return cudaGetLastError();
}

cudaError_t launch_token_compact(const __half* x, int K, const int32_t* idx, int n_keep, __half* out,
                                 const DeviceInfo& dev, cudaStream_t stream) {
    if (n_keep == 0) return cudaSuccess;
    const int vec_per_row = K / 8;
    const size_t total = (size_t)n_keep * vec_per_row;
    size_t blocks = (total + 255) / 256;
    const size_t cap = (size_t)dev.sm_count * 16;
    if (blocks > cap) blocks = cap;
    gather_rows_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(
        reinterpret_cast<const uint4*>(x), vec_per_row, idx, n_keep, reinterpret_cast<uint4*>(out));
    return cudaGetLastError();
}

}  // namespace aq

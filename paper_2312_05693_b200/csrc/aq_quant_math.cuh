// The arithmetic of the activation quantizer (Eq. 1, Eq. 2 / Eq. 5 with zp = 0 and a power-of-two step),
// shared by the quantize kernels and the decode kernel that quantizes its own activations.
#pragma once

#include "aq_common.cuh"

namespace aq {

namespace {

__device__ inline int quantize_one(float v, float inv, float lo, float hi) {
    const float t = v * inv;                 // exact: inv is a power of two
    if (t != t) return 0;                    // NaN
    return (int)fminf(fmaxf(rintf(t), lo), hi);
}

// Eight halves -> eight codes in two 32-bit words, in half2 arithmetic, for exponents whose 2^-e is a
// normal half (|e| <= 14). Every step is exact or rounds exactly like the fp32 route: the product by
// a power of two is exact unless it leaves the half range (overflow saturates to Inf and is clamped
// like any large value; results below 2^-14 round to code 0 either way); NaN is cleared to 0 by a
// lane mask; clamping to the integer bounds before rounding gives the same code as after; adding
// 1536 (ulp 1 in [1024, 2048)) rounds to the nearest integer, ties to even, and leaves the code's
// two's-complement byte in the low 8 bits of the half's bit pattern.
__device__ __forceinline__ void quantize8_half2(const uint4& d, __half2 inv2, __half2 lo2, __half2 hi2, uint32_t& w0,
                                                uint32_t& w1) {
    const __half2* h = reinterpret_cast<const __half2*>(&d);
    const __half2 bias = __floats2half2_rn(1536.0f, 1536.0f);
    uint32_t r[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __half2 t = __hmul2(h[i], inv2);
        const uint32_t ok = __heq2_mask(t, t);                            // 0xFFFF per lane that is not NaN
        uint32_t tb = *reinterpret_cast<uint32_t*>(&t) & ok;
        t = *reinterpret_cast<__half2*>(&tb);
        t = __hadd2(__hmin2(__hmax2(t, lo2), hi2), bias);
        r[i] = *reinterpret_cast<uint32_t*>(&t);
    }
    w0 = __byte_perm(r[0], r[1], 0x6420);
    w1 = __byte_perm(r[2], r[3], 0x6420);
}

// 8 halves -> 8 values in fp32 arithmetic. With TRIP factors (Eq. 5 with a per-channel alpha,
// `al` = the 8 factor bytes of these channels) channel k uses the step 2^(e + alpha_k) and its code
// is stored shifted left by alpha_k, the form in which the factor enters the integer product.
__device__ __forceinline__ uint2 quantize8_fp32(const uint4& d, int e, float lo, float hi, const uint2* al) {
    const __half* h = reinterpret_cast<const __half*>(&d);
    const uint8_t* ab = reinterpret_cast<const uint8_t*>(al);
    uint32_t out[2];
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        uint32_t word = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int i = 4 * w + b;
            const int a = al ? (int)ab[i] : 0;
            const float inv = __int_as_float((127 - e - a) << 23);           // 2^-(e + alpha)
            word |= ((uint32_t)(quantize_one(__half2float(h[i]), inv, lo, hi) << a) & 0xFFu) << (8 * b);
        }
        out[w] = word;
    }
    return make_uint2(out[0], out[1]);
}
}  // namespace

}  // namespace aq

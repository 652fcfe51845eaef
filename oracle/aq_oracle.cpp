// CPU checker for the quantized linear layer of Agile-Quant (arXiv 2312.05693).
//
// TEST INFRASTRUCTURE ONLY. This file is a plain, slow, host-only restatement of
// what the layer computes, written from the paper so that the CUDA library can be
// compared against it. It shares no code with the CUDA library, is never called by
// it, and must not be used as a product path. Every function states the passage of
// the paper it follows; where the paper is silent the reading taken is stated too.
//
// The layer (Sec. 4.4, "Efficient TRIP Matrix Multiplication"): activations are
// quantized layer-wise (one scale for the whole matrix), weights per output channel
// (optionally per 128-wide group of the reduction dimension), the products are
// summed as integers, and the result is mapped back to floating point.
//
// Build: g++ -O3 -march=native -fopenmp -shared -fPIC aq_oracle.cpp -o libaq_oracle.so
// The only parallelism is one OpenMP "parallel for" over output rows.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <algorithm>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

// ---------------------------------------------------------------------------
// IEEE binary16 <-> binary32 / binary64, written from the format's definition
// (1 sign, 5 exponent bits with bias 15, 10 fraction bits).
// ---------------------------------------------------------------------------

// Exact widening: every binary16 value is a binary32 value.
float orc_half_to_float(uint16_t h) {
    const int sign = (h >> 15) & 1;
    const int ex = (h >> 10) & 0x1F;
    const int frac = h & 0x3FF;
    float v;
    if (ex == 0) {
        v = std::ldexp((float)frac, -24);                 // subnormal or zero
    } else if (ex == 31) {
        v = frac ? std::nanf("") : INFINITY;
    } else {
        v = std::ldexp((float)(1024 + frac), ex - 25);    // (1 + frac/1024) * 2^(ex-15)
    }
    return sign ? -v : v;
}

// Round-to-nearest-even narrowing from binary64 with a single rounding.
uint16_t orc_double_to_half(double d) {
    const uint16_t sign = std::signbit(d) ? 0x8000u : 0u;
    if (std::isnan(d)) return (uint16_t)(sign | 0x7E00u);
    double a = std::fabs(d);
    if (std::isinf(a)) return (uint16_t)(sign | 0x7C00u);
    if (a == 0.0) return sign;
    int ex;
    (void)std::frexp(a, &ex);          // a = m * 2^ex, m in [0.5, 1)
    int e = ex - 1;                    // floor(log2 a)
    if (e < -14) e = -14;              // subnormal range shares the spacing of 2^-14
    const double ulp = std::ldexp(1.0, e - 10);
    double r = std::nearbyint(a / ulp);  // division by a power of two is exact; ties to even
    if (r >= 2048.0) { r = 1024.0; e += 1; }
    if (e > 15) return (uint16_t)(sign | 0x7C00u);        // beyond 65504 -> infinity
    const int ri = (int)r;
    if (ri < 1024) return (uint16_t)(sign | ri);          // subnormal (e == -14)
    return (uint16_t)(sign | ((e + 15) << 10) | (ri - 1024));
}

uint16_t orc_float_to_half(float f) { return orc_double_to_half((double)f); }

// ---------------------------------------------------------------------------
// Code range, Eq. 1 (signed set): q in {-2^(b-1), ..., 2^(b-1)-1}.
// ---------------------------------------------------------------------------
static inline int code_min(int bits) { return -(1 << (bits - 1)); }
static inline int code_max(int bits) { return (1 << (bits - 1)) - 1; }

// Round to nearest, ties to even: the paper's rounding bracket in Eq. 2 / Eq. 5 has
// no tie rule; the IEEE default is taken.
static inline float round_half_even(float v) { return std::nearbyintf(v); }

// ---------------------------------------------------------------------------
// Weight quantization. Sec. 4.4 (last paragraph): engines support per-channel
// quantization of the weight matrix; Sec. 5.1: weights are 4-bit. The paper takes
// its 4-bit weights from GPTQ; here they are round-to-nearest, symmetric:
//   a   = max |w| over the channel (or over one 128-wide group of the channel)
//   s   = fp16( a / 7 )             (stored scale; 7 = 2^(4-1)-1, Eq. 1)
//   c   = clip( round(w / s), -8, 7 )   (Eq. 2 with zp = 0 and the signed set)
// An all-zero group gets s = 1; a scale that underflows fp16 gets the smallest
// positive fp16 number. group == 0 means one group spanning all of K.
// codes: int8 [N][K]; scales: fp16 bits [N][G], G = K/group (1 if group == 0).
// ---------------------------------------------------------------------------
void orc_quantize_weights(const uint16_t* w, int N, int K, int group,
                          int8_t* codes, uint16_t* scales) {
    const int gs = group > 0 ? group : K;
    const int G = K / gs;
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < G; ++g) {
            const uint16_t* row = w + (size_t)n * K + (size_t)g * gs;
            float a = 0.0f;
            for (int k = 0; k < gs; ++k) a = std::max(a, std::fabs(orc_half_to_float(row[k])));
            const float s32 = a / 7.0f;
            uint16_t sh = orc_float_to_half(s32);
            if ((sh & 0x7FFF) == 0) sh = (a == 0.0f) ? 0x3C00 /*1.0*/ : 0x0001 /*2^-24*/;
            scales[(size_t)n * G + g] = sh;
            const float s = orc_half_to_float(sh);
            for (int k = 0; k < gs; ++k) {
                float r = round_half_even(orc_half_to_float(row[k]) / s);
                r = std::min(std::max(r, -8.0f), 7.0f);
                codes[(size_t)n * K + (size_t)g * gs + k] = (int8_t)r;
            }
        }
    }
}

// Logical packing used by this checker only: byte j of a row holds code 2j in bits
// 0-3 and code 2j+1 in bits 4-7, two's-complement nibbles. (Sec. 4.4 "INT4
// Multiplier" stores two adjacent weights side by side; which two is a layout
// choice that does not change any result.)
void orc_pack_w4(const int8_t* codes, int N, int K, uint8_t* packed) {
    for (size_t i = 0; i < (size_t)N * K / 2; ++i) {
        const uint8_t lo = (uint8_t)codes[2 * i] & 0xF;
        const uint8_t hi = (uint8_t)codes[2 * i + 1] & 0xF;
        packed[i] = (uint8_t)(lo | (hi << 4));
    }
}

void orc_unpack_w4(const uint8_t* packed, int N, int K, int8_t* codes) {
    for (size_t i = 0; i < (size_t)N * K / 2; ++i) {
        const int lo = packed[i] & 0xF, hi = packed[i] >> 4;
        codes[2 * i] = (int8_t)(lo >= 8 ? lo - 16 : lo);
        codes[2 * i + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
}

// ---------------------------------------------------------------------------
// Token pruning, Eq. 4: X^P = F^P(X) keeps n < m tokens by importance. The scores
// are an input (the paper derives them from attention to the start token, Sec. 4.3).
// Kept: the n_keep largest scores; equal scores are resolved toward the lower
// index; kept indices are returned in ascending order so tokens stay in sequence
// order. Returns 0, or -1 on bad arguments.
// ---------------------------------------------------------------------------
int orc_token_select(const float* scores, int M, int n_keep, int32_t* idx) {
    if (n_keep < 0 || n_keep > M) return -1;
    std::vector<int32_t> order(M);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return scores[a] > scores[b]; });
    std::vector<int32_t> kept(order.begin(), order.begin() + n_keep);
    std::sort(kept.begin(), kept.end());
    std::copy(kept.begin(), kept.end(), idx);
    return 0;
}

void orc_token_compact(const uint16_t* x, int K, const int32_t* idx, int n_keep, uint16_t* out) {
    for (int i = 0; i < n_keep; ++i)
        std::memcpy(out + (size_t)i * K, x + (size_t)idx[i] * K, (size_t)K * sizeof(uint16_t));
}

// ---------------------------------------------------------------------------
// Layer-wise activation scale. Eq. 6 takes the scale from the range of the (pruned)
// activation X^P; Sec. 4.4: all channels share one scale. Reading taken here:
// symmetric (zp = 0), TRIP factor alpha = 0 for every channel, and the scale is the
// power of two 2^e with e the smallest integer such that (2^(b-1)-1) * 2^e >= max|X^P|,
// so nothing clips. max|X^P| == 0 gives e = 0. NaN entries are ignored; an infinite
// maximum is treated as the largest finite fp16 value.
// row_idx == NULL: rows 0..M-1 of x; otherwise rows row_idx[0..M-1].
// ---------------------------------------------------------------------------
int orc_pow2_exponent(float a, int bits) {
    if (!(a > 0.0f)) return 0;
    if (std::isinf(a)) a = 65504.0f;
    const float qmax = (float)code_max(bits);
    int e = 0;
    while (std::ldexp(qmax, e) < a) ++e;
    while (std::ldexp(qmax, e - 1) >= a) --e;
    return e;
}

float orc_absmax(const uint16_t* x, int K, const int32_t* row_idx, int M) {
    float a = 0.0f;
    for (int m = 0; m < M; ++m) {
        const uint16_t* row = x + (size_t)(row_idx ? row_idx[m] : m) * K;
        for (int k = 0; k < K; ++k) {
            const float v = std::fabs(orc_half_to_float(row[k]));
            if (v > a) a = v;   // false for NaN
        }
    }
    return a;
}

int orc_layer_exponent(const uint16_t* x, int K, const int32_t* row_idx, int M, int bits) {
    return orc_pow2_exponent(orc_absmax(x, K, row_idx, M), bits);
}

// ---------------------------------------------------------------------------
// Activation codes. Eq. 2 / Eq. 5 with zp = 0, alpha = 0, s = 2^e and the signed set
// of Eq. 1:  q = clip( round(x / 2^e), -2^(b-1), 2^(b-1)-1 ).
// x / 2^e is exact in binary32 for every fp16 x and every |e| <= 40, so the code is
// uniquely defined. NaN maps to 0. Codes are stored one per int8 also for b = 4.
// ---------------------------------------------------------------------------
void orc_quantize_act(const uint16_t* x, int K, const int32_t* row_idx, int M,
                      int bits, int e, int8_t* q) {
    const float lo = (float)code_min(bits), hi = (float)code_max(bits);
    for (int m = 0; m < M; ++m) {
        const uint16_t* row = x + (size_t)(row_idx ? row_idx[m] : m) * K;
        for (int k = 0; k < K; ++k) {
            const float v = std::ldexp(orc_half_to_float(row[k]), -e);
            float r;
            if (std::isnan(v)) r = 0.0f;
            else r = std::min(std::max(round_half_even(v), lo), hi);
            q[(size_t)m * K + k] = (int8_t)r;
        }
    }
}

// ---------------------------------------------------------------------------
// TRIP factors (Eq. 5 with a per-channel alpha_k, zp = 0, s = 2^e): channel k is quantized with
// the coarser step 2^(e + alpha_k),
//     q = clip( round(x / 2^(e + alpha_k)), -2^(b-1), 2^(b-1)-1 ),
// and enters the integer product as q * 2^alpha_k. Sec. 4.4 moves the factor onto the matching
// weight column; q_k * (c_k * 2^alpha_k) and (q_k * 2^alpha_k) * c_k are the same integer, and
// the second form is what is stored here (one int8 per value). Returns how many values did not
// fit int8 (0 when bits = 4 and alpha <= 4).
// ---------------------------------------------------------------------------
long long orc_quantize_act_trip(const uint16_t* x, int K, const int32_t* row_idx, int M, int bits, int e,
                                const uint8_t* alpha, int8_t* v) {
    const float lo = (float)code_min(bits), hi = (float)code_max(bits);
    long long misfit = 0;
    for (int m = 0; m < M; ++m) {
        const uint16_t* row = x + (size_t)(row_idx ? row_idx[m] : m) * K;
        for (int k = 0; k < K; ++k) {
            const int a = alpha[k];
            const float t = std::ldexp(orc_half_to_float(row[k]), -(e + a));
            int q = 0;
            if (!std::isnan(t)) q = (int)std::min(std::max(round_half_even(t), lo), hi);
            const int val = q * (1 << a);
            if (val < -128 || val > 127) ++misfit;
            v[(size_t)m * K + k] = (int8_t)val;
        }
    }
    return misfit;
}

// Eq. 8, with the clipping of Eq. 5 inside the quantizer (without it the finest step would always
// win): for every channel the alpha in {0..k_max} with the smallest squared reconstruction error
// over the calibration tokens; the smallest alpha among equals. Errors are summed in binary64 over
// tokens in ascending order, product and sum rounded separately (no fused multiply-add), so that
// another implementation following the same order reaches the same decision. Non-finite values
// are skipped.
void orc_trip_calibrate(const uint16_t* x, int K, const int32_t* row_idx, int M, int bits, int e, int k_max,
                        uint8_t* alpha_out) {
    const double lo = (double)code_min(bits), hi = (double)code_max(bits);
    for (int k = 0; k < K; ++k) {
        int best = 0;
        double best_err = 0.0;
        for (int a = 0; a <= k_max; ++a) {
            double err = 0.0;
            for (int m = 0; m < M; ++m) {
                const double xv = (double)orc_half_to_float(x[(size_t)(row_idx ? row_idx[m] : m) * K + k]);
                if (!std::isfinite(xv)) continue;
                const double q = std::min(std::max(std::nearbyint(std::ldexp(xv, -(e + a))), lo), hi);
                const double d = xv - std::ldexp(q, e + a);
                volatile double sq = d * d;            // rounded product, kept apart from the sum
                err = err + sq;
            }
            if (a == 0 || err < best_err) { best = a; best_err = err; }
        }
        alpha_out[k] = (uint8_t)best;
    }
}

// ---------------------------------------------------------------------------
// Integer matrix product (Sec. 4.4; Algorithm 1 computes the same sums of 4-bit
// products in SIMD lanes):  acc[m][n][g] = sum over k in group g of q[m][k]*c[n][k].
// int32 result with an int64 shadow; the return value counts sums that did not fit
// int32 (0 for every supported size). acc: int32 [M][N][G].
// ---------------------------------------------------------------------------
long long orc_int_gemm(const int8_t* q, const int8_t* c, int M, int N, int K, int group,
                       int32_t* acc) {
    const int gs = group > 0 ? group : K;
    const int G = K / gs;
    long long overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            for (int g = 0; g < G; ++g) {
                int64_t s = 0;
                for (int k = g * gs; k < (g + 1) * gs; ++k)
                    s += (int64_t)q[(size_t)m * K + k] * (int64_t)c[(size_t)n * K + k];
                if (s > INT32_MAX || s < INT32_MIN) ++overflow;
                acc[((size_t)m * N + n) * G + g] = (int32_t)s;
            }
        }
    }
    return overflow;
}

// ---------------------------------------------------------------------------
// Mapping back to floating point: y[m][n] = 2^e * sum_g s_w[n][g] * acc[m][n][g],
// evaluated in binary64 with groups in ascending order, rounded once to fp16.
// (The paper's edge kernel requantizes its output for the next operator, Sec. 4.4;
// an fp16 output is what this layer's callers consume.)
// ---------------------------------------------------------------------------
void orc_dequant(const int32_t* acc, const uint16_t* scales, int e, int M, int N, int G,
                 uint16_t* y) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double s = 0.0;
            for (int g = 0; g < G; ++g)
                s += (double)acc[((size_t)m * N + n) * G + g] *
                     (double)orc_half_to_float(scales[(size_t)n * G + g]);
            y[(size_t)m * N + n] = orc_double_to_half(std::ldexp(s, e));
        }
    }
}

// The same two steps for a list of (row, col) output positions, so that full-size
// outputs can be spot-checked without forming the whole product.
void orc_linear_sampled(const int8_t* q, const int8_t* c, const uint16_t* scales, int e,
                        int N, int K, int group, const int32_t* rows, const int32_t* cols,
                        int count, int32_t* acc /*[count][G]*/, uint16_t* y /*[count]*/) {
    const int gs = group > 0 ? group : K;
    const int G = K / gs;
    (void)N;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < count; ++i) {
        const int m = rows[i], n = cols[i];
        double s = 0.0;
        for (int g = 0; g < G; ++g) {
            int64_t a = 0;
            for (int k = g * gs; k < (g + 1) * gs; ++k)
                a += (int64_t)q[(size_t)m * K + k] * (int64_t)c[(size_t)n * K + k];
            acc[(size_t)i * G + g] = (int32_t)a;
            s += (double)a * (double)orc_half_to_float(scales[(size_t)n * G + g]);
        }
        y[i] = orc_double_to_half(std::ldexp(s, e));
    }
}

// ---------------------------------------------------------------------------
// The whole layer in the paper's order: (prune) -> layer scale -> activation codes
// -> integer product -> floating-point output. scale_mode 0: e = e0 - clip_shift
// (clip_shift >= 0 lowers the exponent so outliers saturate); scale_mode 1: e given.
// Any of q_out / acc_out may be NULL. Returns the exponent e through e_out.
// ---------------------------------------------------------------------------
long long orc_linear(const uint16_t* x, int K, const int32_t* row_idx, int M, int bits,
                     int scale_mode, int clip_shift_or_exp, const int8_t* c,
                     const uint16_t* scales, int N, int group, uint16_t* y, int8_t* q_out,
                     int32_t* acc_out, int32_t* e_out) {
    const int gs = group > 0 ? group : K;
    const int G = K / gs;
    const int e = scale_mode == 0 ? orc_layer_exponent(x, K, row_idx, M, bits) - clip_shift_or_exp
                                  : clip_shift_or_exp;
    std::vector<int8_t> qbuf;
    int8_t* q = q_out;
    if (!q) { qbuf.resize((size_t)M * K); q = qbuf.data(); }
    orc_quantize_act(x, K, row_idx, M, bits, e, q);
    std::vector<int32_t> abuf;
    int32_t* acc = acc_out;
    if (!acc) { abuf.resize((size_t)M * N * G); acc = abuf.data(); }
    const long long ovf = orc_int_gemm(q, c, M, N, K, group, acc);
    orc_dequant(acc, scales, e, M, N, G, y);
    if (e_out) *e_out = e;
    return ovf;
}

// ---------------------------------------------------------------------------
// The unsigned quantizer with a zero point, exactly the form of Eq. 2 / Eq. 5-7 (alpha = 0):
//     q = CLIP( round(x / s) + zp, 0, 2^b - 1 ),   zp = CLIP( round(-min / s), 0, 2^b - 1 ),
// with the scale read as a power of two like everywhere else in this file: s = 2^e, e the smallest
// integer with (2^b - 1) * 2^e >= max - min (Eq. 6 with alpha = 0). Readings: the range is widened to
// contain 0 (min' = min(min, 0), max' = max(max, 0)), so that zp is a code; NaN is ignored by min and
// max and maps to the code zp (value 0); +-Inf count as +-65504. Everything is exact in binary64.
// ---------------------------------------------------------------------------
void orc_asym_params(const uint16_t* x, int K, const int32_t* row_idx, int M, int bits, int* e_out, int* zp_out) {
    double lo = 0.0, hi = 0.0;
    for (int m = 0; m < M; ++m) {
        const uint16_t* row = x + (size_t)(row_idx ? row_idx[m] : m) * K;
        for (int k = 0; k < K; ++k) {
            double v = (double)orc_half_to_float(row[k]);
            if (std::isnan(v)) continue;
            if (std::isinf(v)) v = v > 0 ? 65504.0 : -65504.0;
            if (v < lo) lo = v;
            if (v > hi) hi = v;
        }
    }
    const double range = hi - lo, qr = (double)((1 << bits) - 1);
    int e = 0;
    if (range > 0.0) {
        while (std::ldexp(qr, e) < range) ++e;
        while (std::ldexp(qr, e - 1) >= range) --e;
    }
    const double zp = std::min(std::max(std::nearbyint(std::ldexp(-lo, -e)), 0.0), qr);
    *e_out = e;
    *zp_out = (int)zp;
}

// Unsigned codes of Eq. 2 for given e and zp, one per byte.
void orc_quantize_act_asym(const uint16_t* x, int K, const int32_t* row_idx, int M, int bits, int e, int zp,
                           uint8_t* q) {
    const double qr = (double)((1 << bits) - 1);
    for (int m = 0; m < M; ++m) {
        const uint16_t* row = x + (size_t)(row_idx ? row_idx[m] : m) * K;
        for (int k = 0; k < K; ++k) {
            const double v = (double)orc_half_to_float(row[k]);
            double r = (double)zp;
            if (!std::isnan(v)) r = std::min(std::max(std::nearbyint(std::ldexp(v, -e)) + (double)zp, 0.0), qr);
            q[(size_t)m * K + k] = (uint8_t)r;
        }
    }
}

// The layer with such codes: y[m][n] = fp16( 2^e * sum_g s_w[n][g] * sum_{k in g} (q[m][k] - zp) * c[n][k] ),
// integer sums exact (int64), the rest in binary64 with one rounding to fp16. acc (may be NULL):
// the integer sums [M][N][G].
void orc_linear_asym(const uint8_t* q, int zp, const int8_t* c, const uint16_t* scales, int e, int M, int N, int K,
                     int group, long long* acc /*[M][N][G] or NULL*/, uint16_t* y) {
    const int gs = group > 0 ? group : K;
    const int G = K / gs;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            double s = 0.0;
            for (int g = 0; g < G; ++g) {
                long long a = 0;
                for (int k = g * gs; k < (g + 1) * gs; ++k)
                    a += (long long)((int)q[(size_t)m * K + k] - zp) * (long long)c[(size_t)n * K + k];
                if (acc) acc[((size_t)m * N + n) * G + g] = a;
                s += (double)a * (double)orc_half_to_float(scales[(size_t)n * G + g]);
            }
            y[(size_t)m * N + n] = orc_double_to_half(std::ldexp(s, e));
        }
    }
}

// ---------------------------------------------------------------------------
// Log2 quantizer, Eq. 3 (used for the softmax output, Sec. 5.1):
//     Q(x|b) = Sign(x) * CLIP( round( -log2( |x| / max|X| ) ), 0, 2^(b-1) - 1 ),
// i.e. x is represented by Sign(x) * max|X| * 2^-k. Readings: the maximum is taken over the whole
// tensor (layer-wise, like every activation scale here); Sign(0) = 0 makes the value 0, which needs a
// code of its own, so the stored int8 is Sign(x) * (k + 1) and 0 stands for an exact zero; NaN is
// ignored by the maximum and stored as 0; +-Inf count as +-65504. The rounding is decided in binary64:
// every boundary 2^-(k+1/2) is irrational, no ratio of two halves comes closer to one than about 2^-24
// relative, far more than the error of log2 in binary64.
// Returns the maximum (as a float; 0 for an all-zero tensor, in which case every code is 0).
// ---------------------------------------------------------------------------
float orc_log2_quantize(const uint16_t* x, long long count, int bits, int8_t* codes) {
    double mx = 0.0;
    for (long long i = 0; i < count; ++i) {
        double v = std::fabs((double)orc_half_to_float(x[i]));
        if (std::isnan(v)) continue;
        if (std::isinf(v)) v = 65504.0;
        if (v > mx) mx = v;
    }
    const double kmax = (double)((1 << (bits - 1)) - 1);
    for (long long i = 0; i < count; ++i) {
        double v = (double)orc_half_to_float(x[i]);
        if (std::isnan(v) || v == 0.0 || mx == 0.0) { codes[i] = 0; continue; }
        if (std::isinf(v)) v = v > 0 ? 65504.0 : -65504.0;
        const double k = std::min(std::max(std::nearbyint(-std::log2(std::fabs(v) / mx)), 0.0), kmax);
        codes[i] = (int8_t)((v > 0 ? 1 : -1) * ((int)k + 1));
    }
    return (float)mx;
}

// Attention-times-value with such codes (Sec. 5.1; "shift-only" products): P [H][M][J] as log2 codes
// with maximum p_max, V [H][J][D] as int8 codes with the layer exponent e_v:
//     acc[h][m][d] = sum_j Sign_j * ( Vq[h][j][d] * 2^(kmax - k_j) )            (exact integers)
//     y[h][m][d]   = fp16( p_max * 2^(e_v - kmax) * acc[h][m][d] )               (one rounding)
void orc_attn_v_log2(const int8_t* pcodes, float p_max, const int8_t* vq, int e_v, int H, int M, int J, int D,
                     int bits, long long* acc_out /* or NULL */, uint16_t* y) {
    const int kmax = (1 << (bits - 1)) - 1;
#pragma omp parallel for schedule(static)
    for (int hm = 0; hm < H * M; ++hm) {
        const int h = hm / M;
        const int8_t* prow = pcodes + (size_t)hm * J;
        for (int d = 0; d < D; ++d) {
            long long a = 0;
            for (int j = 0; j < J; ++j) {
                const int c = prow[j];
                if (c == 0) continue;
                const int k = (c > 0 ? c : -c) - 1;
                const long long term = (long long)vq[((size_t)h * J + j) * D + d] * (1LL << (kmax - k));
                a += c > 0 ? term : -term;
            }
            if (acc_out) acc_out[(size_t)hm * D + d] = a;
            y[(size_t)hm * D + d] = orc_double_to_half(std::ldexp((double)p_max * (double)a, e_v - kmax));
        }
    }
}

// Progressive pruning ratio, Eq. 9: gamma = 1 - (1 - beta)^(1/m).
double orc_progressive_ratio(double beta, int m) { return 1.0 - std::pow(1.0 - beta, 1.0 / m); }

int orc_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

}  // extern "C"

// Log2 quantization of the softmax output (paper Eq. 3, Sec. 5.1) and the attention-times-value
// product on its codes, where every product is a shift of the int8 value code.
#include <cuda.h>

#include "aq_common.cuh"

namespace aq {

namespace {

// ---- layer-wide max |x| as an fp16 bit pattern (NaN ignored, Inf counts as 65504) -------------
// 16-byte loads where the pointer allows; the first thread also takes the ragged tail.
__global__ void __launch_bounds__(256)
log2_absmax_kernel(const __half* __restrict__ x, long long count, Control* __restrict__ ctl) {
    unsigned int b = 0;
    auto take = [&](unsigned int hb) {
        hb &= 0x7FFFu;
        if (hb > 0x7C00u) return;
        if (hb == 0x7C00u) hb = 0x7BFFu;
        b = max(b, hb);
    };
    const bool vec = (reinterpret_cast<uintptr_t>(x) & 15u) == 0;
    const long long nvec = vec ? count / 8 : 0;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    // two values per instruction: the half2 maximum returns the other operand when one is NaN, so NaN
    // never enters; Inf does and is replaced by the largest finite value below
    __half2 m2 = __float2half2_rn(0.0f);
#pragma unroll 4
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
        const uint4 d = __ldg(xv + i);
        const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint32_t a = w[t] & 0x7FFF7FFFu;
            m2 = __hmax2(m2, *reinterpret_cast<const __half2*>(&a));
        }
    }
    {
        const uint32_t mw = *reinterpret_cast<const uint32_t*>(&m2);
        take(mw & 0xFFFFu);
        take(mw >> 16);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (long long i = nvec * 8; i < count; ++i) take(__half_as_ushort(x[i]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xFFFFFFFFu, b, o));
    if ((threadIdx.x & 31) == 0 && b != 0) atomicMax(&ctl->absmax_bits, b);
}

// A positive fp16 bit pattern as mant * 2^expo with 1024 <= mant < 2048.
__device__ __forceinline__ void half_parts(unsigned int hb, int& mant, int& expo) {
    const int ex = (int)(hb >> 10), fr = (int)(hb & 0x3FFu);
    if (ex > 0) { mant = 1024 + fr; expo = ex - 25; }
    else {                                         // subnormal: fr * 2^-24, fr > 0
        const int sh = __clz(fr) - 21;             // brings the leading one to bit 10
        mant = fr << sh;
        expo = -24 - sh;
    }
}

// Eq. 3: k = clip(round(-log2(|x| / max)), 0, kmax), stored as Sign(x) * (k + 1), 0 for zero / NaN.
// The rounding is decided with integers: -log2(r) = (Eb - Ea) + log2(mb / ma), and log2(mb / ma) passes
// +-1/2 exactly when mb^2 passes 2 ma^2 or ma^2 / 2 (mantissas are 11-bit integers).
// The two mantissa thresholds of the rounding rule for a given maximum mantissa mb (1024..2047):
// t_up = largest ma with 2 ma^2 <= mb^2 (below or at it k rounds up), t_down = smallest ma with
// ma^2 > 2 mb^2 (from it on k rounds down).
__device__ __forceinline__ void log2_thresholds(int mb, int& t_up, int& t_down) {
    int a = (int)(sqrtf(0.5f * (float)mb * (float)mb));
    while (2 * (a + 1) * (a + 1) <= mb * mb) ++a;
    while (2 * a * a > mb * mb) --a;
    t_up = a;
    int b = (int)(sqrtf(2.0f * (float)mb * (float)mb));
    while (b * b > 2 * mb * mb) --b;
    while ((b + 1) * (b + 1) <= 2 * mb * mb) ++b;
    t_down = b + 1;
}

__device__ __forceinline__ int log2_code(unsigned int raw, unsigned int mb_bits, int eb, int t_up, int t_down, int kmax) {
    unsigned int hb = raw & 0x7FFFu;
    const bool none = hb == 0 || hb > 0x7C00u || mb_bits == 0;      // zero, NaN, or an all-zero layer
    hb = min(hb, 0x7BFFu);                                           // Inf counts as the largest finite value
    // Without branches (softmax outputs mix normal and subnormal values inside every warp): the exact
    // conversion to binary32 normalises subnormals, |x| = (1024 + top ten fraction bits) * 2^(E - 10).
    const unsigned int fb = __float_as_uint(__half2float(__ushort_as_half((unsigned short)hb)));
    const int ma = 1024 + (int)((fb >> 13) & 0x3FFu);
    const int ea = (int)(fb >> 23) - 137;
    int k = eb - ea + (ma <= t_up ? 1 : 0) - (ma >= t_down ? 1 : 0);
    k = min(max(k, 0), kmax) + 1;
    return none ? 0 : ((raw & 0x8000u) ? -k : k);
}

// codes -> weights: c > 0 -> 128 >> (c - 1); 0 -> 0; a negative code is not representable here:
// it is recorded in the status word (11) and treated as 0.
__device__ __forceinline__ uint32_t log2_factors4(uint32_t c4, bool& bad) {
    uint32_t o = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int c = (int)(int8_t)((c4 >> (8 * t)) & 0xFFu);
        bad |= c < 0;
        o |= (c > 0 ? (128u >> (c - 1)) : 0u) << (8 * t);
    }
    return o;
}

// 4-bit codes in half2 arithmetic. k does not increase with |x|, so k = #{ j in 1..7 : |x| < B_j } with B_j the
// smallest half whose k is below j. By the integer rule above, k <= j - 1 needs, at exponent Eb - j, a mantissa
// from t_down on, and at exponent Eb - j + 1 a mantissa above t_up; one exponent lower nothing qualifies, one
// higher everything does. So B_j = t_down * 2^(Eb - j) when t_down is a mantissa (<= 2047), else
// (t_up + 1) * 2^(Eb - j + 1), rounded up to a half where it falls between subnormals (the inputs are halves,
// so that keeps the comparison's outcome). Seven compares and adds for two elements replace the exponent and
// mantissa arithmetic per element.
struct Log2Fast {
    __half2 bound[7];
};
__device__ __forceinline__ Log2Fast log2_fast_bounds(int mb, int eb, int t_up, int t_down) {
    Log2Fast f;
#pragma unroll
    for (int j = 1; j <= 7; ++j) {
        const float b = t_down <= 2047 ? ldexpf((float)t_down, eb - j) : ldexpf((float)max(t_up + 1, 1024), eb - j + 1);
        f.bound[j - 1] = __half2half2(__float2half_ru(b));
    }
    (void)mb;
    return f;
}
// Two halves -> (k + 1) * valid as halves (codes), or 2^(7 - k) * valid (factors); valid = 0 for zero and NaN.
template <bool FACTORS>
__device__ __forceinline__ __half2 log2_fast2(__half2 x2, const Log2Fast& f) {
    const __half2 mag = __habs2(x2);
    const __half2 valid = __hgt2(mag, __float2half2_rn(0.0f));                // 1 or 0; NaN compares false
    const __half2 ax = __hmin2(mag, __float2half2_rn(65504.0f));              // Inf counts as the largest finite value (a NaN lane becomes 65504 here and is dropped by valid)
    __half2 r = __float2half2_rn(FACTORS ? 128.0f : 1.0f);
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        const __half2 below = __hlt2(ax, f.bound[j]);                         // 1 or 0
        if (FACTORS) r = __hfma2(below, __float2half2_rn(-(float)(64 >> j)), r);   // 128 - 64 - 32 - ... = 2^(7 - k)
        else r = __hadd2(r, below);
    }
    return __hmul2(r, valid);
}

__global__ void __launch_bounds__(256)
log2_codes_kernel(const __half* __restrict__ x, long long count, int bits, Control* __restrict__ ctl,
                  int8_t* __restrict__ codes, uint32_t* __restrict__ max_bits_out, int as_factors) {
    // as_factors (4-bit codes of a non-negative input): instead of the code c the byte 2^(kmax - k) = 128 >> (c - 1)
    // is written (0 for a zero), the form the tensor-core product takes; a negative value is reported (status 11)
    bool bad = false;
    const unsigned int mb_bits = ctl->absmax_bits;
    if (blockIdx.x == 0 && threadIdx.x == 0 && max_bits_out) *max_bits_out = mb_bits;
    const int kmax = (1 << (bits - 1)) - 1;
    int mb = 1024, eb = 0, t_up = 0, t_down = 0;
    if (mb_bits) half_parts(mb_bits, mb, eb);
    log2_thresholds(mb, t_up, t_down);
    const bool vec = (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && (reinterpret_cast<uintptr_t>(codes) & 7u) == 0;
    const long long nvec = vec ? count / 8 : 0;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    if (bits == 4 && mb_bits != 0) {
        const Log2Fast fast = log2_fast_bounds(mb, eb, t_up, t_down);
#pragma unroll 4
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
            const uint4 d = __ldg(xv + i);
            const uint32_t w[4] = {d.x, d.y, d.z, d.w};
            uint32_t m[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const __half2 x2 = *reinterpret_cast<const __half2*>(&w[t]);
                __half2 r;
                if (as_factors) {
                    r = log2_fast2<true>(x2, fast);
                    // a negative input has no factor: recorded, its byte is 0
                    const __half2 neg = __hlt2(x2, __float2half2_rn(0.0f));
                    bad |= (*reinterpret_cast<const uint32_t*>(&neg) != 0u);
                    r = __hfma2(neg, __hneg2(r), r);                                    // r * (1 - neg)
                    r = __hadd2(r, __float2half2_rn(1024.0f));                           // the integer sits in the low bits
                } else {
                    r = log2_fast2<false>(x2, fast);
                    uint32_t rb = *reinterpret_cast<uint32_t*>(&r) | (w[t] & 0x80008000u);   // Sign(x) * (k + 1)
                    r = __hadd2(*reinterpret_cast<__half2*>(&rb), __float2half2_rn(1536.0f));   // two's complement in the low byte
                }
                m[t] = *reinterpret_cast<uint32_t*>(&r);
            }
            *reinterpret_cast<uint2*>(codes + 8 * i) = make_uint2(__byte_perm(m[0], m[1], 0x6420), __byte_perm(m[2], m[3], 0x6420));
        }
    } else
#pragma unroll 4
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (long long)gridDim.x * blockDim.x) {
        const uint4 d = __ldg(xv + i);
        const uint32_t w[4] = {d.x, d.y, d.z, d.w};
        uint32_t out[2] = {0u, 0u};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const uint32_t c0 = (uint32_t)log2_code(w[t] & 0xFFFFu, mb_bits, eb, t_up, t_down, kmax) & 0xFFu;
            const uint32_t c1 = (uint32_t)log2_code(w[t] >> 16, mb_bits, eb, t_up, t_down, kmax) & 0xFFu;
            out[t >> 1] |= (c0 | (c1 << 8)) << (16 * (t & 1));
        }
        if (as_factors) { out[0] = log2_factors4(out[0], bad); out[1] = log2_factors4(out[1], bad); }
        *reinterpret_cast<uint2*>(codes + 8 * i) = make_uint2(out[0], out[1]);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (long long i = nvec * 8; i < count; ++i) {
            const int c = log2_code(__half_as_ushort(x[i]), mb_bits, eb, t_up, t_down, kmax);
            bad |= as_factors && c < 0;
            codes[i] = as_factors ? (int8_t)(uint8_t)(c > 0 ? (128u >> (c - 1)) : 0u) : (int8_t)c;
        }
    if (bad) atomicCAS(&ctl->status, 0u, 11u);
}

// ---- attention x value on the codes -----------------------------------------------------------
// A CTA of 256 threads takes `rows` consecutive query rows of one head and all D value columns; a
// thread owns one row and four consecutive columns (one 4-byte load of value codes per j) and adds
// each value code shifted left by kmax - k_j, negated for negative probabilities, skipped for zeros.
__global__ void __launch_bounds__(256)
attn_v_log2_kernel(const int8_t* __restrict__ pcodes, const uint32_t* __restrict__ max_bits,
                   const int8_t* __restrict__ vq, const int32_t* __restrict__ e_v, int M, int J, int D, int bits,
                   int rows, __half* __restrict__ y, int32_t* __restrict__ acc_dump) {
    const int quads = D / 4;
    const int r = threadIdx.x / quads, dq = threadIdx.x % quads;
    const int h = blockIdx.y;
    const int m = blockIdx.x * rows + r;
    if (r >= rows || m >= M) return;
    const int kmax = (1 << (bits - 1)) - 1;
    const int8_t* prow = pcodes + ((size_t)h * M + m) * J;
    const char4* vcol = reinterpret_cast<const char4*>(vq + (size_t)h * J * D) + dq;
    int a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll 4
    for (int j = 0; j < J; ++j) {
        const int c = prow[j];
        if (c == 0) continue;
        const char4 v = __ldg(vcol + (size_t)j * quads);
        const int sh = kmax + 1 - abs(c);
        const int sg = c > 0 ? 1 : -1;
        a0 += (sg * (int)v.x) << sh;
        a1 += (sg * (int)v.y) << sh;
        a2 += (sg * (int)v.z) << sh;
        a3 += (sg * (int)v.w) << sh;
    }
    const float pmax = __half2float(__ushort_as_half((unsigned short)(*max_bits & 0xFFFFu)));
    const float scale = pmax * __int_as_float((127 + *e_v - kmax) << 23);
    const size_t o = ((size_t)h * M + m) * D + 4 * dq;
    y[o + 0] = __float2half_rn(scale * (float)a0);
    y[o + 1] = __float2half_rn(scale * (float)a1);
    y[o + 2] = __float2half_rn(scale * (float)a2);
    y[o + 3] = __float2half_rn(scale * (float)a3);
    if (acc_dump) { acc_dump[o] = a0; acc_dump[o + 1] = a1; acc_dump[o + 2] = a2; acc_dump[o + 3] = a3; }
}

// ---- the same product on the tensor cores (non-negative P, i.e. a softmax output) --------------
// With P >= 0 the factor 2^(kmax - k) is an unsigned byte (1..128), so the product is a plain
// u8 x s8 -> s32 contraction over the key index j: acc[m][d] = sum_j w[m][j] * v[d][j], with both
// operands stored j-major. tcgen05.mma kind::i8 reads both from shared memory (128-byte swizzle,
// staged by TMA); the accumulator [128 query rows x D] lives in tensor memory.

// [H][J][D] int8 -> [H][D][J] int8 through a 32 x 32 shared-memory tile.
__global__ void __launch_bounds__(256)
transpose_i8_kernel(const int8_t* __restrict__ in, int J, int D, int8_t* __restrict__ out) {
    __shared__ int8_t tile[32][33];
    const int h = blockIdx.z, j0 = blockIdx.x * 32, d0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;          // 32 x 8
    for (int r = ty; r < 32; r += 8) {
        const int j = j0 + r, d = d0 + tx;
        tile[r][tx] = (j < J && d < D) ? in[((size_t)h * J + j) * D + d] : (int8_t)0;
    }
    __syncthreads();
    for (int r = ty; r < 32; r += 8) {
        const int d = d0 + r, j = j0 + tx;
        if (d < D && j < J) out[((size_t)h * D + d) * J + j] = tile[tx][r];
    }
}

// The same through a 64 x 64 tile with 4-byte accesses on both sides (D and J multiples of 4, 4-byte aligned
// buffers): a warp reads and writes 64-byte row pieces as words instead of 32 single bytes.
__global__ void __launch_bounds__(256)
transpose_i8_words_kernel(const int8_t* __restrict__ in, int J, int D, int8_t* __restrict__ out) {
    __shared__ __align__(4) int8_t tile[64][68];                      // [j][d], rows padded to 68 bytes
    const int h = blockIdx.z, j0 = blockIdx.x * 64, d0 = blockIdx.y * 64;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int idx = (int)threadIdx.x + 256 * k, r = idx >> 4, c = 4 * (idx & 15);
        const int j = j0 + r, d = d0 + c;
        uint32_t w = 0u;
        if (j < J && d < D) w = *reinterpret_cast<const uint32_t*>(in + ((size_t)h * J + j) * D + d);
        *reinterpret_cast<uint32_t*>(&tile[r][c]) = w;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int idx = (int)threadIdx.x + 256 * k, r = idx >> 4, c = 4 * (idx & 15);      // output row d0 + r, columns j0 + c..
        const int d = d0 + r, j = j0 + c;
        if (d < D && j < J) {
            const uint32_t w = (uint32_t)(uint8_t)tile[c][r] | ((uint32_t)(uint8_t)tile[c + 1][r] << 8) |
                               ((uint32_t)(uint8_t)tile[c + 2][r] << 16) | ((uint32_t)(uint8_t)tile[c + 3][r] << 24);
            *reinterpret_cast<uint32_t*>(out + ((size_t)h * D + d) * J + j) = w;
        }
    }
}

constexpr int kTcStages = 4;
// warp 0: TMA, warp 1: MMA + TMEM owner, then EW epilogue warps (4, or 8: two per quarter of the tensor-memory lanes,
// each taking half of the columns, for products with one k step per tile, where the epilogue sets the pace)
constexpr int kConvWarps = 8;                        // warps that turn codes into byte factors (CONVERT)
constexpr int tc_threads(int ew, bool convert = false) { return (2 + ew + (convert ? kConvWarps : 0)) * 32; }
constexpr unsigned long long kTcWaitCycles = 4000000000ull;

__device__ __forceinline__ uint32_t a_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool a_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(a_smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; false when the limit ran out or another role gave up.
__device__ __forceinline__ bool a_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
    if (a_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!a_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag) return false;
            if ((unsigned long long)(clock64() - t0) > kTcWaitCycles) { *abort_flag = 12u; return false; }
        }
    }
    return true;
}
// K-major tile with 128-byte rows written by TMA with the 128-byte swizzle (see aq_gemm_tensor.cu).
__device__ __forceinline__ uint64_t a_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

template <int DN, int RT, int EW>
struct AttnSmem {
    alignas(1024) uint8_t a[kTcStages][RT * 128 * 128];   // weights tile: RT x 128 query rows x 128 j
    alignas(1024) uint8_t b[kTcStages][DN * 128];    // value tile: DN columns x 128 j
    // Output staging: each epilogue warp owns two boxes of 32 rows x 64 halves (128-byte rows, written
    // with the 128-byte swizzle of the store's tensor map), for alternate 64-column chunks.
    alignas(1024) uint8_t ystage[EW][2][32 * 128];
    alignas(8) uint64_t full[kTcStages];
    uint64_t empty[kTcStages];
    uint64_t conv[kTcStages];                        // CONVERT: the A tile of the stage holds byte factors -> MMA
    uint64_t acc_full[2];                            // MMA -> epilogue, one per accumulator stage
    uint64_t acc_empty[2];                           // epilogue (4 warps) -> MMA
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
};

// Batched int8 contraction y[h][m][n] = scale * sum_k A[h*M + m][k] * B[h*NB + n][k] (both operands
// k-major). A work item is (128 rows of A, head): all tiles of DN rows of B for those rows. The grid is
// persistent: CTA c takes the items c, c + gridDim.x, ..., and the ring of operand stages and the two
// accumulator stages in tensor memory run on across items, so the producer fetches the next item's tiles
// while the epilogue of the last tile of this one still writes (a CTA's 16 k steps of one item alone were
// mostly fill and drain). With RT = 2 an item is 256 rows of A, two accumulators of 128 rows that share
// every tile of B: what limits this kernel is the L2 -> SM path, and the B tile is then fetched once for
// twice the rows. A is unsigned or signed bytes, B signed. CONVERT: A arrives as 4-bit log2 codes (c = k + 1,
// 0 for a zero) and kConvWarps more warps turn every landed A tile into byte factors 128 >> k in place before the
// MMA reads it, so that attention x value needs no conversion pass over the probabilities in memory.
// scale = (max_bits ? the half in its low 16 bits : 1) * 2^(*e1 + (e2 ? *e2 : 0) + e_off).
// Used for attention x value (A = byte factors of the log2 codes, B = transposed value codes, k = key
// index) and for the query x key product (A, B = int8 codes, k = head dimension).
template <int DN, bool A_SIGNED, int RT = 1, int EW = 4, bool CONVERT = false>
__global__ void __launch_bounds__(tc_threads(EW, CONVERT), 1)
attn_v_tc_kernel(const __grid_constant__ CUtensorMap a_map, const __grid_constant__ CUtensorMap b_map,
                 const __grid_constant__ CUtensorMap y_map, const uint32_t* __restrict__ max_bits, const int32_t* __restrict__ e1, const int32_t* __restrict__ e2,
                 int e_off, int H, int M, int J /* length of k */, int NB, __half* __restrict__ y, Control* __restrict__ ctl) {
    extern __shared__ uint8_t attn_smem_raw[];
    using Smem = AttnSmem<DN, RT, EW>;
    static_assert(EW == 4 || (EW == 8 && DN % 64 == 0), "epilogue warps: one or two per lane quarter");
    constexpr int kColsPerWarp = DN / (EW / 4);                          // columns an epilogue warp drains
    static_assert(2 * RT * DN <= 512, "two accumulator stages of RT x DN columns in tensor memory");
    constexpr int kRows = RT * 128;                                       // rows of A per item
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(attn_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int MT = (M + kRows - 1) / kRows;                               // row tiles per head
    const int items = MT * H;                                             // work items; item w = (head w / MT, row tile w % MT)
    const int JB = (J + 127) / 128;
    const int NT = (NB + DN - 1) / DN;                                    // tiles of B rows per item
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTcStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(a_smem_u32(&sm.full[s])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(a_smem_u32(&sm.empty[s])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a_smem_u32(&sm.conv[s])), "r"(kConvWarps) : "memory");
        }
        for (int a = 0; a < 2; ++a) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(a_smem_u32(&sm.acc_full[a])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a_smem_u32(&sm.acc_empty[a])), "r"(EW) : "memory");
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(a_smem_u32(&sm.tmem_base)), "r"((uint32_t)(2 * RT * DN)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm.tmem_base;
    volatile uint32_t* abort_flag = &sm.abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;                                                   // stages filled so far, over all items
            bool ok = true;
            for (int w = blockIdx.x; w < items && ok; w += gridDim.x) {
              const int h = w / MT, m0 = (w % MT) * kRows;
              for (int i = 0; i < NT * JB; ++i, ++it) {
                const int nt = i / JB, jb = i % JB, n0 = nt * DN;
                const int s = it % kTcStages;
                if (!a_wait(&sm.empty[s], ((it / kTcStages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                             ::"r"(a_smem_u32(&sm.full[s])), "r"((uint32_t)((kRows + DN) * 128)) : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                    ::"r"(a_smem_u32(sm.a[s])), "l"(&a_map), "r"(jb * 128), "r"(h * M + m0), "r"(a_smem_u32(&sm.full[s]))
                    : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                    ::"r"(a_smem_u32(sm.b[s])), "l"(&b_map), "r"(jb * 128), "r"(h * NB + n0), "r"(a_smem_u32(&sm.full[s]))
                    : "memory");
              }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // D = s32 (2 at bits 4-5), A unsigned 8-bit (0 at bits 7-9), B signed 8-bit (1 at bits 10-12),
            // both K-major, N >> 3 at bits 17-22, M >> 4 at bits 24-28
            constexpr uint32_t idesc = (2u << 4) | ((A_SIGNED ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(DN >> 3) << 17) |
                                       ((uint32_t)(128 >> 4) << 24);
            bool ok = true;
            int it = 0, tc = 0;                                           // stages and tiles consumed so far, over all items
            for (int w = blockIdx.x; w < items && ok; w += gridDim.x)
            for (int nt = 0; nt < NT && ok; ++nt, ++tc) {
              const int a = tc & 1;
              ok = a_wait(&sm.acc_empty[a], ((tc >> 1) & 1) ^ 1, abort_flag);      // the epilogue has drained this stage
              if (!ok) break;
              for (int jb = 0; jb < JB && ok; ++jb, ++it) {
                const int s = it % kTcStages;
                ok = a_wait(CONVERT ? &sm.conv[s] : &sm.full[s], (it / kTcStages) & 1, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t adesc = a_desc_sw128(a_smem_u32(sm.a[s]));
                const uint64_t bdesc = a_desc_sw128(a_smem_u32(sm.b[s]));
#pragma unroll
                for (int r = 0; r < RT; ++r) {
                    // the r-th 128 rows of the A tile start 16 KB (1024 in descriptor units of 16 bytes) further on
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const uint32_t accumulate = (jb == 0 && t == 0) ? 0u : 1u;
                        asm volatile(
                            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                            ::"r"(tmem + (uint32_t)((a * RT + r) * DN)), "l"(adesc + (uint64_t)(1024 * r + 2 * t)),
                              "l"(bdesc + (uint64_t)(2 * t)), "r"(idesc), "r"(accumulate)
                            : "memory");
                    }
                }
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(a_smem_u32(&sm.empty[s])) : "memory");
              }
              if (ok)
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(a_smem_u32(&sm.acc_full[a])) : "memory");
            }
        }
    } else if (CONVERT && warp >= 2 + EW) {
        // ---- codes -> byte factors, in place, on every A tile that has landed (the map is bytewise, so the
        // tile's swizzle does not matter). Per 32-bit word: a byte permute looks the factors of codes 1..7 up
        // by the codes' low three bits, code 8 (k = 7) is added as 1, codes above 8 and negative codes give 0,
        // and a negative code is recorded (status 11) as the conversion pass does.
        const int cw = warp - (2 + EW);                                       // 0..kConvWarps-1
        bool bad = false;
        int it = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < items && ok; w += gridDim.x) {
            for (int i = 0; i < NT * JB && ok; ++i, ++it) {
                const int s = it % kTcStages;
                ok = __all_sync(0xFFFFFFFFu, a_wait(&sm.full[s], (it / kTcStages) & 1, abort_flag) ? 1 : 0) != 0;
                if (!ok) break;
                uint4* tile = reinterpret_cast<uint4*>(sm.a[s]);
#pragma unroll 4
                for (int v = cw * 32 + lane; v < kRows * 128 / 16; v += kConvWarps * 32) {
                    uint4 c = tile[v];
                    uint32_t* cwds = reinterpret_cast<uint32_t*>(&c);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const uint32_t x = cwds[t];
                        const uint32_t neg = x & 0x80808080u;
                        const uint32_t x7 = x & 0x7F7F7F7Fu;
                        const uint32_t big = (x7 + 0x77777777u) & 0x80808080u;          // bytes from 9 up
                        const uint32_t low = x & 0x07070707u;
                        const uint32_t sel = __byte_perm(low | (low >> 4), 0u, 0x4420);   // four 3-bit indices as nibbles
                        uint32_t r = __byte_perm(0x20408000u, 0x02040810u, sel);          // index 0..7 -> 0, 128, 64, ..., 2
                        r |= (x7 >> 3) & 0x01010101u;                                     // code 8 -> 1 (9..15 are cleared below)
                        const uint32_t kill = ((neg | big) >> 7) * 0xFFu;
                        cwds[t] = r & ~kill;
                        bad |= neg != 0u;
                    }
                    tile[v] = c;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes before the tensor core's reads
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_smem_u32(&sm.conv[s])) : "memory");
            }
        }
        if (bad) atomicCAS(&ctl->status, 0u, 11u);
    } else {
        const int quarter = warp & 3;                                     // TMEM lanes this warp may read
        const float pmax = max_bits ? __half2float(__ushort_as_half((unsigned short)(*max_bits & 0xFFFFu))) : 1.0f;
        const float scale = pmax * __int_as_float((127 + *e1 + (e2 ? *e2 : 0) + e_off) << 23);
        int tc = 0;                                                       // tiles drained so far, over all items
        bool alive = true;
        for (int w = blockIdx.x; w < items && alive; w += gridDim.x) {
          const int h = w / MT, m0_item = (w % MT) * kRows;
          for (int nt = 0; nt < NT; ++nt, ++tc) {
            const int a = tc & 1, n0 = nt * DN;
            if (!(__all_sync(0xFFFFFFFFu, a_wait(&sm.acc_full[a], (tc >> 1) & 1, abort_flag) ? 1 : 0) != 0)) { alive = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int ew = warp - 2;
#pragma unroll 1
            for (int r = 0; r < RT; ++r) {
            const int m0 = m0_item + r * 128, m = m0 + quarter * 32 + lane;          // this accumulator's 128 rows
#pragma unroll 1
            for (int c0 = ((warp - 2) >> 2) * kColsPerWarp; c0 < (((warp - 2) >> 2) + 1) * kColsPerWarp; c0 += 32) {
                uint32_t v[32];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                      "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                      "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                      "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((a * RT + r) * DN + c0))
                    : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                // 32 columns of this thread's row -> 64 bytes of its 128-byte staging row; 16-byte chunk j of
                // row r sits at chunk position j ^ (r & 7), as the store's tensor map expects
                const int row0 = m0 + quarter * 32;
                if (row0 + 32 > M) {
                    // a box of 32 rows would run into the next head's rows: this warp stores its rows itself
                    if (m < M) {
                        __half* yrow = y + ((size_t)h * M + m) * NB + n0;
#pragma unroll
                        for (int q8 = 0; q8 < 4; ++q8) {
                            if (n0 + c0 + 8 * q8 >= NB) break;               // NB is a multiple of 8
                            __half2 o[4];
#pragma unroll
                            for (int t = 0; t < 4; ++t)
                                o[t] = __floats2half2_rn(scale * (float)(int)v[8 * q8 + 2 * t], scale * (float)(int)v[8 * q8 + 2 * t + 1]);
                            *reinterpret_cast<uint4*>(yrow + c0 + 8 * q8) = *reinterpret_cast<uint4*>(o);
                        }
                    }
                    continue;
                }
                const int box = (c0 >> 6) & 1, half_of_box = (c0 >> 5) & 1;
                uint8_t* srow = sm.ystage[ew][box] + lane * 128;
                if (half_of_box == 0) {
                    // the box is about to be rewritten: the store that used it last must have read it (with two
                    // boxes in rotation one younger store may still be pending)
                    if (lane == 0) {
                        if (kColsPerWarp > 64) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    }
                    __syncwarp();
                }
#pragma unroll
                for (int q8 = 0; q8 < 4; ++q8) {
                    __half2 o[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        o[t] = __floats2half2_rn(scale * (float)(int)v[8 * q8 + 2 * t], scale * (float)(int)v[8 * q8 + 2 * t + 1]);
                    const int chunk = half_of_box * 4 + q8;
                    *reinterpret_cast<uint4*>(srow + ((chunk ^ (lane & 7)) << 4)) = *reinterpret_cast<uint4*>(o);
                }
                if (half_of_box == 1 || c0 + 32 >= DN) {   // (a warp's column range ends on a box boundary or at DN)
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    const int col = n0 + (c0 & ~63);
                    if (lane == 0 && col < NB) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&y_map), "r"(col), "r"(h * M + row0), "r"(a_smem_u32(sm.ystage[ew][box])) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            }
            }
            // this warp's part of the accumulator stage is in registers / written: hand the stage back
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a_smem_u32(&sm.acc_empty[a])) : "memory");
          }
        }
    }
    if (warp >= 2 && warp < 2 + EW && lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // staging rows live until read
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (sm.abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);                   // let copies in flight land
        if (threadIdx.x == 0) atomicCAS(&ctl->status, 0u, sm.abort_flag);
    }
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)(2 * RT * DN)) : "memory");
}

typedef CUresult (*AttnEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <int DN, bool A_SIGNED, int RT = 1, int EW = 4, bool CONVERT = false>
cudaError_t launch_attn_tc(const void* w, const int8_t* vt, const uint32_t* max_bits, const int32_t* e1, const int32_t* e2,
                           int e_off, int H, int M, int J, int NB, __half* y, Control* ctl, const DeviceInfo& dev,
                           cudaStream_t stream) {
    using Smem = AttnSmem<DN, RT, EW>;
    const size_t smem_bytes = sizeof(Smem) + 1024;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(attn_v_tc_kernel<DN, A_SIGNED, RT, EW, CONVERT>, dev.device, smem_bytes); e != cudaSuccess)
        return e;
    CUtensorMap amap, bmap;
    const cuuint32_t estr[2] = {1u, 1u};
    const cuuint64_t strides[1] = {(cuuint64_t)J};
    const cuuint64_t adims[2] = {(cuuint64_t)J, (cuuint64_t)H * M};
    const cuuint32_t abox[2] = {128u, (cuuint32_t)(RT * 128)};
    const cuuint64_t bdims[2] = {(cuuint64_t)J, (cuuint64_t)H * NB};
    const cuuint32_t bbox[2] = {128u, (cuuint32_t)DN};
    AttnEncodeFn enc = reinterpret_cast<AttnEncodeFn>(dev.encode_tiled);
    if (enc(&amap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(w), adims, strides, abox, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    if (enc(&bmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(vt), bdims, strides, bbox, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    // outputs: [H*M rows][NB] halves, stored in boxes of 64 columns x 32 rows with the 128-byte swizzle
    CUtensorMap ymap;
    const cuuint64_t ydims[2] = {(cuuint64_t)NB, (cuuint64_t)H * M};
    const cuuint64_t ystrides[1] = {(cuuint64_t)NB * 2};
    const cuuint32_t ybox[2] = {64u, 32u};
    if (enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, ydims, ystrides, ybox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    const int items = ((M + RT * 128 - 1) / (RT * 128)) * H;
    dim3 grid(items < dev.sm_count ? items : dev.sm_count);
    attn_v_tc_kernel<DN, A_SIGNED, RT, EW, CONVERT><<<grid, tc_threads(EW, CONVERT), smem_bytes, stream>>>(amap, bmap, ymap, max_bits, e1, e2, e_off, H, M,
                                                                            J, NB, y, ctl);
    return cudaGetLastError();
}

}  // namespace

size_t attn_tc_scratch_bytes(int H, int M, int J, int D) {
    (void)M;
    return ((size_t)H * D * J + 255) / 256 * 256;
}

// scratch: the transposed value codes, H*D*J bytes.
// p_is_factors: pcodes already holds the byte factors (written by the log2 kernel); otherwise the product kernel
// converts the codes tile by tile in shared memory.
cudaError_t launch_attn_v_log2_tc(const int8_t* pcodes, const uint32_t* max_bits, const int8_t* vq, const int32_t* e_v,
                                  int H, int M, int J, int D, __half* y, Control* ctl, void* scratch,
                                  const DeviceInfo& dev, cudaStream_t stream, bool p_is_factors) {
    int8_t* vt = static_cast<int8_t*>(scratch);
    cudaError_t e = cudaSuccess;
    // codes or byte factors: the product kernel reads either
    const uint8_t* w = reinterpret_cast<const uint8_t*>(pcodes);
    if (J % 4 == 0 && D % 4 == 0 && (reinterpret_cast<uintptr_t>(vq) & 3u) == 0 && (reinterpret_cast<uintptr_t>(vt) & 3u) == 0)
        transpose_i8_words_kernel<<<dim3((J + 63) / 64, (D + 63) / 64, H), 256, 0, stream>>>(vq, J, D, vt);
    else
        transpose_i8_kernel<<<dim3((J + 31) / 32, (D + 31) / 32, H), 256, 0, stream>>>(vq, J, D, vt);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const bool wide_items = M % 256 == 0;       // items of 256 query rows share every value tile; whole items only
    if (p_is_factors)
        return D == 64 ? launch_attn_tc<64, false>(w, vt, max_bits, e_v, nullptr, -7, H, M, J, D, y, ctl, dev, stream)
               : wide_items ? launch_attn_tc<128, false, 2>(w, vt, max_bits, e_v, nullptr, -7, H, M, J, D, y, ctl, dev, stream)
                            : launch_attn_tc<128, false>(w, vt, max_bits, e_v, nullptr, -7, H, M, J, D, y, ctl, dev, stream);
    return D == 64 ? launch_attn_tc<64, false, 1, 4, true>(w, vt, max_bits, e_v, nullptr, -7, H, M, J, D, y, ctl, dev, stream)
           : wide_items ? launch_attn_tc<128, false, 2, 4, true>(w, vt, max_bits, e_v, nullptr, -7, H, M, J, D, y, ctl, dev, stream)
                        : launch_attn_tc<128, false, 1, 4, true>(w, vt, max_bits, e_v, nullptr, -7, H, M, J, D, y, ctl, dev, stream);
}

// Query x key: s[h][m][j] = 2^(e_q + e_k) * sum_d q[h][m][d] * k[h][j][d], int8 codes, D = 128.
cudaError_t launch_attn_qk_tc(const int8_t* qc, const int32_t* e_q, const int8_t* kc, const int32_t* e_k, int H, int M,
                              int J, int D, __half* s_out, Control* ctl, const DeviceInfo& dev, cudaStream_t stream) {
    // one k step per tile (k = D = 128): the epilogue, 64 KB of scores per tile and row block, sets the pace
    return launch_attn_tc<128, true, 1, 8>(qc, kc, nullptr, e_q, e_k, 0, H, M, D, J, s_out, ctl, dev, stream);
}

cudaError_t launch_log2_quantize(const __half* x, long long count, int bits, Control* ctl, int8_t* codes,
                                 uint32_t* max_bits_out, const DeviceInfo& dev, cudaStream_t stream, bool as_factors) {
    long long blocks = (count / 8 + 255) / 256;
    const long long cap = (long long)dev.sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    log2_absmax_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(x, count, ctl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    log2_codes_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(x, count, bits, ctl, codes, max_bits_out, as_factors ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_attn_v_log2(const int8_t* pcodes, const uint32_t* max_bits, const int8_t* vq, const int32_t* e_v,
                               int H, int M, int J, int D, int bits, __half* y, int32_t* acc_dump, cudaStream_t stream) {
    const int quads = D / 4;
    const int rows = 256 / quads;                  // D <= 1024 and D % 4 == 0 are checked by the caller
    dim3 grid((M + rows - 1) / rows, H);
    attn_v_log2_kernel<<<grid, 256, 0, stream>>>(pcodes, max_bits, vq, e_v, M, J, D, bits, rows, y, acc_dump);
    return cudaGetLastError();
}

}  // namespace aq

// Log2 quantization of the softmax output (paper Eq. 3, Sec. 5.1) and the attention-times-value
// product on its codes, where every product is a shift of the int8 value code.
#include "aq_common.cuh"

namespace aq {

namespace {

// ---- layer-wide max |x| as an fp16 bit pattern (NaN ignored, Inf counts as 65504) -------------
__global__ void __launch_bounds__(256)
log2_absmax_kernel(const __half* __restrict__ x, long long count, Control* __restrict__ ctl) {
    unsigned int b = 0;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        unsigned int hb = __half_as_ushort(x[i]) & 0x7FFFu;
        if (hb > 0x7C00u) continue;
        if (hb == 0x7C00u) hb = 0x7BFFu;
        b = max(b, hb);
    }
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
__global__ void __launch_bounds__(256)
log2_codes_kernel(const __half* __restrict__ x, long long count, int bits, const Control* __restrict__ ctl,
                  int8_t* __restrict__ codes, uint32_t* __restrict__ max_bits_out) {
    const unsigned int mb_bits = ctl->absmax_bits;
    if (blockIdx.x == 0 && threadIdx.x == 0 && max_bits_out) *max_bits_out = mb_bits;
    const int kmax = (1 << (bits - 1)) - 1;
    int mb = 1024, eb = 0;
    if (mb_bits) half_parts(mb_bits, mb, eb);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        const unsigned int raw = __half_as_ushort(x[i]);
        unsigned int hb = raw & 0x7FFFu;
        int c = 0;
        if (hb != 0 && hb <= 0x7C00u && mb_bits != 0) {
            if (hb == 0x7C00u) hb = 0x7BFFu;
            int ma, ea;
            half_parts(hb, ma, ea);
            int k = eb - ea;
            if (mb * mb >= 2 * ma * ma) k += 1;
            else if (2 * mb * mb < ma * ma) k -= 1;
            k = min(max(k, 0), kmax);
            c = (raw & 0x8000u) ? -(k + 1) : (k + 1);
        }
        codes[i] = (int8_t)c;
    }
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

}  // namespace

cudaError_t launch_log2_quantize(const __half* x, long long count, int bits, Control* ctl, int8_t* codes,
                                 uint32_t* max_bits_out, const DeviceInfo& dev, cudaStream_t stream) {
    long long blocks = (count + 255) / 256;
    const long long cap = (long long)dev.sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    log2_absmax_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(x, count, ctl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    log2_codes_kernel<<<(unsigned int)blocks, 256, 0, stream>>>(x, count, bits, ctl, codes, max_bits_out);
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

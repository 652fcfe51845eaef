// Integer product for few rows (M <= 16 per CTA pass): a weight-streaming reduction on
// CUDA cores. Every packed weight byte is read from HBM exactly once per 16 activation
// rows; products use dp4a (4 int8 x int8 per instruction) on weights widened to 16*code.
// Computes the sums of Sec. 4.4 / Algorithm 1 and the floating-point output.
#include "aq_common.cuh"

namespace aq {

namespace {

constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecPrefetch = 4;      // 128-k blocks in flight per warp (4 x 16 B per lane each)

// CTA = 32 output channels (one lane each) x all of K, K split over the 8 warps by 128-k
// block; grid.y walks the rows in chunks of MB.
template <int MB, bool GROUPED>
__global__ void __launch_bounds__(kDecThreads)
gemm_decode_kernel(const int8_t* __restrict__ q, int M, int K, int N, int Npad,
                   const uint8_t* __restrict__ w_packed, const __half* __restrict__ w_scales,
                   const int32_t* __restrict__ scale_exp, __half* __restrict__ y,
                   int32_t* __restrict__ acc_dump) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int KB = K / kTileK;
    const int n0 = blockIdx.x * 32;
    const int nt = n0 / kTileN, r = (n0 % kTileN) + lane;
    const int n = n0 + lane;
    const int m0 = blockIdx.y * MB;
    const uint8_t* wbase = w_packed + (size_t)nt * KB * kBlockBytes + (size_t)r * 16;

    int acc[MB];
    float fsum[MB];
#pragma unroll
    for (int m = 0; m < MB; ++m) { acc[m] = 0; fsum[m] = 0.0f; }

    const int T = KB > warp ? (KB - warp + kDecWarps - 1) / kDecWarps : 0;
    uint4 buf[kDecPrefetch][4];
#pragma unroll
    for (int d = 0; d < kDecPrefetch; ++d) {
        if (d < T) {
            const uint8_t* p = wbase + (size_t)(warp + d * kDecWarps) * kBlockBytes;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                buf[d][j] = __ldg(reinterpret_cast<const uint4*>(p + j * kTileN * 16));
        }
    }
    for (int t0 = 0; t0 < T; t0 += kDecPrefetch) {
#pragma unroll
        for (int d = 0; d < kDecPrefetch; ++d) {
            const int t = t0 + d;
            if (t >= T) break;
            const int kb = warp + t * kDecWarps;
            uint4 cur[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) cur[j] = buf[d][j];
            if (t + kDecPrefetch < T) {
                const uint8_t* p = wbase + (size_t)(kb + kDecPrefetch * kDecWarps) * kBlockBytes;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    buf[d][j] = __ldg(reinterpret_cast<const uint4*>(p + j * kTileN * 16));
            }
            if (GROUPED) {
#pragma unroll
                for (int m = 0; m < MB; ++m) acc[m] = 0;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t w[4] = {cur[j].x, cur[j].y, cur[j].z, cur[j].w};
                uint32_t w8[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    w8[2 * i] = (w[i] << 4) & 0xF0F0F0F0u;       // 16*code for k0..k0+3
                    w8[2 * i + 1] = w[i] & 0xF0F0F0F0u;          // 16*code for k0+4..k0+7
                }
#pragma unroll
                for (int m = 0; m < MB; ++m) {
                    if (m0 + m < M) {
                        const uint4* xp = reinterpret_cast<const uint4*>(
                            q + (size_t)(m0 + m) * K + kb * kTileK + 32 * j);
                        const uint4 x0 = __ldg(xp), x1 = __ldg(xp + 1);
                        int a = acc[m];
                        a = __dp4a((int)w8[0], (int)x0.x, a);
                        a = __dp4a((int)w8[1], (int)x0.y, a);
                        a = __dp4a((int)w8[2], (int)x0.z, a);
                        a = __dp4a((int)w8[3], (int)x0.w, a);
                        a = __dp4a((int)w8[4], (int)x1.x, a);
                        a = __dp4a((int)w8[5], (int)x1.y, a);
                        a = __dp4a((int)w8[6], (int)x1.z, a);
                        a = __dp4a((int)w8[7], (int)x1.w, a);
                        acc[m] = a;
                    }
                }
            }
            if (GROUPED) {
                const float s = __half2float(w_scales[(size_t)kb * Npad + n]);
#pragma unroll
                for (int m = 0; m < MB; ++m) {
                    const int a = acc[m] >> 4;                   // exact: sums are multiples of 16
                    fsum[m] = fmaf((float)a, s, fsum[m]);
                    if (acc_dump && m0 + m < M && n < N)
                        acc_dump[((size_t)(m0 + m) * N + n) * KB + kb] = a;
                }
            }
        }
    }

    // cross-warp reduction: integers when one scale spans K, floats otherwise
    __shared__ int red[kDecWarps][MB][32];
#pragma unroll
    for (int m = 0; m < MB; ++m)
        red[warp][m][lane] = GROUPED ? __float_as_int(fsum[m]) : acc[m];
    __syncthreads();
    const float pe = __int_as_float((127 + *scale_exp) << 23);   // 2^e
    for (int m = warp; m < MB; m += kDecWarps) {
        if (m0 + m >= M || n >= N) continue;
        float out;
        if (GROUPED) {
            float s = 0.0f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) s += __int_as_float(red[w][m][lane]);
            out = s * pe;
        } else {
            int s = 0;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) s += red[w][m][lane];
            s >>= 4;
            if (acc_dump) acc_dump[(size_t)(m0 + m) * N + n] = s;
            out = (float)s * __half2float(w_scales[n]) * pe;
        }
        y[(size_t)(m0 + m) * N + n] = __float2half_rn(out);
    }
}

template <int MB>
cudaError_t launch_mb(const GemmArgs& a, cudaStream_t stream) {
    const int Npad = round_up(a.N, kTileN);
    dim3 grid(Npad / 32, (a.M + MB - 1) / MB);
    if (a.group)
        gemm_decode_kernel<MB, true><<<grid, kDecThreads, 0, stream>>>(
            a.q, a.M, a.K, a.N, Npad, a.w_packed, a.w_scales, a.scale_exp, a.y, a.acc_dump);
    else
        gemm_decode_kernel<MB, false><<<grid, kDecThreads, 0, stream>>>(
            a.q, a.M, a.K, a.N, Npad, a.w_packed, a.w_scales, a.scale_exp, a.y, a.acc_dump);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm_decode(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    (void)dev;
    if (a.M <= 1) return launch_mb<1>(a, stream);
    if (a.M <= 2) return launch_mb<2>(a, stream);
    if (a.M <= 4) return launch_mb<4>(a, stream);
    if (a.M <= 8) return launch_mb<8>(a, stream);
    return launch_mb<16>(a, stream);
}

}  // namespace aq

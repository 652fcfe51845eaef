// Offline weight quantization and packing (4-bit, per output channel or per 128-wide
// group; paper Sec. 4.4 last paragraph and Sec. 5.1), and the inverse of the packing.
#include "aq_common.cuh"

namespace aq {

namespace {

__device__ inline float block_max_128(float v, float* red) {
    // 128 threads = 4 warps
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    const float r = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    return r;
}

// Stored scale for a group whose largest magnitude is a: fp16(a/7); 1 for an all-zero
// group; the smallest positive fp16 when a/7 underflows.
__device__ inline __half group_scale(float a) {
    __half s = __float2half_rn(__fdiv_rn(a, 7.0f));
    if ((__half_as_ushort(s) & 0x7FFFu) == 0)
        s = __ushort_as_half(a == 0.0f ? (unsigned short)0x3C00u : (unsigned short)0x0001u);
    return s;
}

// One CTA of 128 threads per (padded) output channel.
__global__ void __launch_bounds__(128)
pack_w4_kernel(const __half* __restrict__ w, int N, int K, int group, uint8_t* __restrict__ packed,
               __half* __restrict__ scales) {
    __shared__ float red[4];
    __shared__ int8_t codes[kTileK];
    const int n = blockIdx.x;
    const int Npad = gridDim.x;
    const int KB = k_blocks(K);
    const int t = threadIdx.x;
    const int nt = n / kTileN, r = n % kTileN;
    const bool live = n < N;
    const __half* row = w + (size_t)n * K;

    float s_row = 1.0f;
    if (group == 0) {
        float a = 0.0f;
        if (live)
            for (int k = t; k < K; k += 128) a = fmaxf(a, fabsf(__half2float(row[k])));
        a = block_max_128(a, red);
        const __half sh = group_scale(a);
        if (t == 0) scales[n] = live ? sh : __ushort_as_half((unsigned short)0);
        s_row = __half2float(sh);
    }
    for (int kb = 0; kb < KB; ++kb) {
        const float wv = (live && kb * kTileK + t < K) ? __half2float(row[kb * kTileK + t]) : 0.0f;   // k >= K: zero codes
        float s = s_row;
        if (group != 0) {
            const float a = block_max_128(fabsf(wv), red);
            const __half sh = group_scale(a);
            if (t == 0) scales[(size_t)kb * Npad + n] = live ? sh : __ushort_as_half((unsigned short)0);
            s = __half2float(sh);
        }
        float c = rintf(__fdiv_rn(wv, s));
        c = fminf(fmaxf(c, -8.0f), 7.0f);
        codes[t] = (int8_t)(int)c;
        __syncthreads();
        if (t < 16) {
            const int j = t >> 2, i = t & 3;
            const int8_t* c8 = codes + 32 * j + 8 * i;
            uint32_t word = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                word |= ((uint32_t)c8[b] & 0xFu) << (8 * b);
                word |= ((uint32_t)c8[4 + b] & 0xFu) << (8 * b + 4);
            }
            *reinterpret_cast<uint32_t*>(packed + packed_unit_offset(KB, nt, kb, j, r) + 4 * i) = word;
        }
        __syncthreads();
    }
}

__global__ void unpack_w4_kernel(const uint8_t* __restrict__ packed, int N, int K,
                                 int8_t* __restrict__ codes) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K) return;
    const int n = (int)(idx / K), k = (int)(idx % K);
    const int KB = k_blocks(K);
    const int kb = k / kTileK, kl = k % kTileK;
    const int j = kl >> 5, i = (kl & 31) >> 3, p = kl & 7;
    const uint8_t byte = packed[packed_unit_offset(KB, n / kTileN, kb, j, n % kTileN) + 4 * i + (p & 3)];
    const int nib = (p & 4) ? (byte >> 4) : (byte & 0xF);
    codes[idx] = (int8_t)(nib >= 8 ? nib - 16 : nib);
}

// One thread per channel: the sum of its codes in every group, times the group's scale, in binary64.
__global__ void weight_offsets_kernel(const uint8_t* __restrict__ packed, const __half* __restrict__ scales, int N,
                                      int K, int group, float* __restrict__ r_out) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    const int KB = k_blocks(K), Npad = round_up(N, kTileN);
    const int nt = n / kTileN, r = n % kTileN;
    double total = 0.0;
    long long run = 0;
    for (int kb = 0; kb < KB; ++kb) {
        int colsum = 0;
        for (int j = 0; j < 4; ++j) {
            const uint4 d = *reinterpret_cast<const uint4*>(packed + packed_unit_offset(KB, nt, kb, j, r));
            const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int b = 0; b < 8; ++b) {
                    const int nib = (w[i] >> (4 * b)) & 0xF;
                    colsum += nib >= 8 ? nib - 16 : nib;
                }
        }
        if (group) total += (double)colsum * (double)__half2float(scales[(size_t)kb * Npad + n]);
        else run += colsum;
    }
    if (!group) total = (double)run * (double)__half2float(scales[n]);
    r_out[n] = (float)total;
}

// Packed storage of 4-bit activation codes: byte j of a row holds code 2j in bits 0-3 and code 2j+1 in
// bits 4-7 (two's-complement nibbles). One thread turns 16 codes into 8 bytes or back.
__global__ void __launch_bounds__(256)
act4_pack_kernel(const uint4* __restrict__ q, size_t n16, uint2* __restrict__ out) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n16) return;
    const uint4 c = q[i];
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
    uint32_t r[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t t = w[k] & 0x0F0F0F0Fu;       // low nibble of every code
        r[k] = t | (t >> 4);                         // bytes 0 and 2 now hold the two pairs of this word
    }
    out[i] = make_uint2(__byte_perm(r[0], r[1], 0x6420), __byte_perm(r[2], r[3], 0x6420));
}

__global__ void __launch_bounds__(256)
act4_unpack_kernel(const uint2* __restrict__ p, size_t n16, uint4* __restrict__ q) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n16) return;
    const uint2 b = p[i];
    const uint32_t w[2] = {b.x, b.y};
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        uint32_t lo = w[k] & 0x0F0F0F0Fu, hi = (w[k] >> 4) & 0x0F0F0F0Fu;
        // sign extension inside each byte: bit 3 set -> bits 4-7 set (8 * 30 = 0xF0, no carry between bytes)
        lo |= (lo & 0x08080808u) * 0x1Eu;
        hi |= (hi & 0x08080808u) * 0x1Eu;
        o[2 * k] = __byte_perm(lo, hi, 0x5140);      // codes 0..3 of this word's 8: lo0 hi0 lo1 hi1
        o[2 * k + 1] = __byte_perm(lo, hi, 0x7362);  // codes 4..7: lo2 hi2 lo3 hi3
    }
    q[i] = make_uint4(o[0], o[1], o[2], o[3]);
}

}  // namespace

cudaError_t launch_act4_pack(const int8_t* q, size_t count, uint8_t* out, cudaStream_t stream) {
    const size_t n16 = count / 16;
    if (n16 == 0) return cudaSuccess;
    act4_pack_kernel<<<(unsigned int)((n16 + 255) / 256), 256, 0, stream>>>(reinterpret_cast<const uint4*>(q), n16,
                                                                          reinterpret_cast<uint2*>(out));
    return cudaGetLastError();
}

cudaError_t launch_act4_unpack(const uint8_t* packed, size_t count, int8_t* q, cudaStream_t stream) {
    const size_t n16 = count / 16;
    if (n16 == 0) return cudaSuccess;
    act4_unpack_kernel<<<(unsigned int)((n16 + 255) / 256), 256, 0, stream>>>(reinterpret_cast<const uint2*>(packed), n16,
                                                                            reinterpret_cast<uint4*>(q));
    return cudaGetLastError();
}

cudaError_t launch_weight_offsets(const uint8_t* packed, const __half* scales, int N, int K, int group, float* r,
                                  cudaStream_t stream) {
    weight_offsets_kernel<<<(N + 127) / 128, 128, 0, stream>>>(packed, scales, N, K, group, r);
    return cudaGetLastError();
}

cudaError_t launch_pack_w4(const __half* w, int N, int K, int group, uint8_t* packed, __half* scales,
                           cudaStream_t stream) {
    const int Npad = round_up(N, kTileN);
    pack_w4_kernel<<<Npad, 128, 0, stream>>>(w, N, K, group, packed, scales);
    return cudaGetLastError();
}

cudaError_t launch_unpack_w4(const uint8_t* packed, int N, int K, int8_t* codes, cudaStream_t stream) {
    const size_t total = (size_t)N * K;
    const unsigned int blocks = (unsigned int)((total + 255) / 256);
    unpack_w4_kernel<<<blocks, 256, 0, stream>>>(packed, N, K, codes);
    return cudaGetLastError();
}

}  // namespace aq

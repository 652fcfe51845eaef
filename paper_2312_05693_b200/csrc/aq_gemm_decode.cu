// Integer product for few rows (M <= 16 per pass): weight-streaming reductions that read
// every packed weight byte from HBM once per 16 activation rows. They compute the sums of
// Sec. 4.4 / Algorithm 1 and the floating-point output.
//
// Two kernels:
//  * a general one (per-group scales, or any M when forced): a CTA owns 32 output channels
//    (one lane each), its 8 warps split K by 128-k block, products use dp4a on weights
//    widened to 16*code, warps meet in shared memory;
//  * a streaming one for one scale per channel and M <= 16: a thread-block cluster shares a
//    128-channel tile and splits K; in each CTA a producer thread streams 8 KB packed blocks
//    and their activation codes into a shared-memory ring with TMA, eight consumer warps
//    multiply (dp4a for one row, the warp-level int8 MMA above). Every CTA keeps the sums over
//    its k range in its own shared memory; the cluster meets once, and every CTA then finishes a
//    slice of the tile's channels by reading the other CTAs' sums over distributed shared memory
//    (integer addition is exact in any order). No workspace, no atomics.
#include <cooperative_groups.h>
#include <cuda.h>

#include "aq_common.cuh"
#include "aq_quant_math.cuh"

namespace cg = cooperative_groups;

namespace aq {

namespace {

constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecPrefetch = 4;      // 128-k blocks in flight per warp (4 x 16 B per lane each)

// Chaining: the code the next layer's quantizer gives the fp16 output value (static exponent; NaN -> 0).
__device__ __forceinline__ int next_code(__half hv, float inv, float lo, float hi) {
    const float t = __half2float(hv) * inv;                 // exact: inv is a power of two
    if (t != t) return 0;
    return (int)fminf(fmaxf(rintf(t), lo), hi);
}

// Chaining: a warp's codes of one token (lane = consecutive channels) are stored one byte each or, packed,
// the even lane stores its code and its neighbour's in one byte of q4 [M][N/2]. All 32 lanes call this
// together; `valid` lanes (the same for a lane pair) store.
__device__ __forceinline__ void store_next_code(int8_t* q_next, size_t index, int code, int packed, bool valid, int lane) {
    if (packed) {
        const int hi = __shfl_down_sync(0xFFFFFFFFu, code, 1);
        if (valid && !(lane & 1)) reinterpret_cast<uint8_t*>(q_next)[index >> 1] = (uint8_t)((code & 0xF) | (hi << 4));
    } else if (valid) {
        q_next[index] = (int8_t)code;
    }
}

// CTA = 32 output channels (one lane each) x all of K, K split over the 8 warps by 128-k
// block; grid.y walks the rows in chunks of MB.
template <int MB, bool GROUPED>
__global__ void __launch_bounds__(kDecThreads)
gemm_decode_kernel(const int8_t* __restrict__ q, int M, int K, int N, int Npad,
                   const uint8_t* __restrict__ w_packed, const __half* __restrict__ w_scales,
                   const int32_t* __restrict__ scale_exp, __half* __restrict__ y,
                   int32_t* __restrict__ acc_dump, Control* __restrict__ ctl, const float* __restrict__ chan_offset,
                   int8_t* __restrict__ q_next, float next_inv, float next_lo, float next_hi, int clear_status,
                   int next_packed) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // this kernel has no bounded waits; after a quantize kernel of the same call the word is that kernel's
    if (clear_status && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) ctl->status = 0;
    const int KB = k_blocks(K);
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
                if (kb * kTileK + 32 * j >= K) break;            // a last block padded with zero codes (K % 128 != 0)
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
        if (m0 + m >= M) continue;                               // the same for the whole warp
        const bool n_ok = n < N;
        const float off = chan_offset && n_ok ? chan_offset[n] : 0.0f;
        float out;
        if (GROUPED) {
            float s = 0.0f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) s += __int_as_float(red[w][m][lane]);
            out = (s + off) * pe;
        } else {
            int s = 0;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) s += red[w][m][lane];
            s >>= 4;
            if (acc_dump && n_ok) acc_dump[(size_t)(m0 + m) * N + n] = s;
            out = fmaf((float)s, n_ok ? __half2float(w_scales[n]) : 0.0f, off) * pe;
        }
        const __half hv = __float2half_rn(out);
        if (q_next)
            store_next_code(q_next, (size_t)(m0 + m) * N + n, next_code(hv, next_inv, next_lo, next_hi), next_packed, n_ok, lane);
        else if (n_ok)
            y[(size_t)(m0 + m) * N + n] = hv;
    }
}

// ---------------------------------------------------------------------------------------
// Streaming kernel (one scale per channel, M <= 16)
// ---------------------------------------------------------------------------------------
constexpr unsigned long long kStrWaitCycles = 4000000000ull;
constexpr int kFuseMaxBlocks = 64;        // k blocks per CTA up to which a single row is quantized inside the product kernel

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool str_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(s_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; false when the limit ran out or another thread of the CTA already gave up.
__device__ __forceinline__ bool str_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
    if (str_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!str_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag) return false;
            if ((unsigned long long)(clock64() - t0) > kStrWaitCycles) { *abort_flag = 1; return false; }
        }
    }
    return true;
}

// One row uses dp4a with one lane per channel; more rows use the warp-level int8 MMA
// (m16n8k32) on 16 rows, with the activation tile stored 128-byte swizzled so that fragment
// loads are free of bank conflicts.
// Ring depth 8 (64 KB of weights in flight per CTA, two CTAs per SM): 9 stages for 16 rows and 12 for one
// row, which shared memory would allow, measured no faster.
// Producer lanes: a wait, an expect and two copies per block are four shared-memory-pipe instructions of a
// hundred cycles and more each next to the working consumers, so one lane cannot issue faster than a block
// per ~500 cycles, which bounds a CTA that streams alone on its SM. With two lanes of the warp in lockstep
// (lane l takes the blocks l, l + 2, ... of the k range) the single-row kernel gains 0.3-1.1 us per launch;
// four lanes gain no more, eight lose, and with 16 rows (tensor-map copies of the codes) two lanes measured
// 0.1-0.3 us slower than one.
template <int MB> struct StreamCfg {
    static constexpr bool kUseMma = MB > 4;
    static constexpr int kRows = kUseMma ? 16 : MB;
    static constexpr int kStages = 8;
    static constexpr int kProdLanes = kUseMma ? 1 : 2;
    // Consumer warps: a channel quarter each, kPhases warps per quarter taking the k blocks in turn. A third
    // warp per quarter measured slower with 16 rows (7.6 / 11.4 / 13.6 -> 8.5 / 12.0 / 14.4 us on the 13B
    // shapes) although a warp holds a block for 600-700 cycles there: the stream slows with the amount of
    // consumer work in flight, not with the time a block waits (with the consumers' arithmetic taken out the
    // same launches take 6.6 / 9.1 / 10.1 us, and the ring is never full either way).
    static constexpr int kPhases = 2;
    // Two CTAs per SM for both routes. Three single-row CTAs would fit (with 128-byte instead of 1024-byte
    // alignment slack), so that under the stable-weights promise the next launch's CTAs sit, fetching, beside
    // two CTAs of this one; measured slower (M = 1 layer 5.8 / 9.1 / 9.7 -> 6.6 / 9.7 / 11.8 us): what the
    // early CTAs fetch is taken from the grid that has to finish first.
    static constexpr int kConsumerWarps = 4 * kPhases;
    static constexpr int kThreads = (1 + kConsumerWarps) * 32;
};

template <int MB, bool WIDE = false>
struct StreamSmem {
    static constexpr int kRows = StreamCfg<MB>::kRows;
    static constexpr int kStages = StreamCfg<MB>::kStages;
    alignas(1024) int8_t x[kStages][kRows * kTileK];       // activation codes of the unit's k block
    alignas(128) uint8_t w[kStages][kBlockBytes];          // packed weight block of the unit
    // this CTA's sums over its k range; rows padded by 8 words so that the MMA route's fragment owners (eight
    // rows at the same columns) spread over the banks
    static constexpr int kSumStride = kTileN + 8;
    alignas(16) int sum[kRows][kSumStride];
    // one row quantized by the kernel itself: the codes of this CTA's k range (up to kFuseMaxBlocks blocks)
    alignas(16) int8_t xq[MB == 1 ? kFuseMaxBlocks * kTileK : 16];
    unsigned int warp_max[StreamCfg<MB>::kThreads / 32];
    // the other CTAs' sums for this CTA's channel slice, by sender: `split` slots of 128 / split channels, or
    // (clusters of 5 to 8) eight slots of 32
    static constexpr int kRecvStride = WIDE ? 256 : kTileN;
    alignas(16) int recv[kRows][kRecvStride];
    alignas(8) uint64_t full[kStages];
    uint64_t empty[kStages];
    volatile uint32_t abort_flag;
};

struct StreamParams {
    int M, K, N, Npad;
    const int8_t* q;
    const uint8_t* w_packed;
    const __half* w_scales;
    const int32_t* scale_exp;
    __half* y;
    int32_t* acc_dump;
    Control* ctl;
    const float* chan_offset;
    int8_t* q_next;
    float next_inv, next_lo, next_hi;
    int clear_status;
    int early_weights;             // the first ring of weight copies may be issued before the wait for the kernel ahead
    int early_dependents;          // the launch behind this one may be set up from this kernel's start
    int next_packed;
    // FUSEQ (one row): the activations themselves; the kernel finds the layer scale, writes the codes of
    // its k range to shared memory (and, from the first channel tile, to q_out) and fills the control block
    const __half* x_row;           // the row's K halves
    const int32_t* row_idx;        // NULL or one index: the row is x_row + row_idx[0] * K
    int8_t* q_out;                 // [K] codes
    int bits, scale_mode, clip_shift_or_exp;
};

// grid = (split, channel tiles), cluster = (split, 1, 1): the CTAs of a cluster share a channel
// tile and take consecutive k ranges; CTA r adds up and writes its slice of the tile's channels:
// [r, r+1) * 128 / split for split 1, 2, 4; WIDE (split 5 to 8, 16-row route only) the groups of four
// channels [32 r / split, 32 (r + 1) / split).
template <int MB, bool FUSEQ = false, bool WIDE = false>
__global__ void __launch_bounds__(StreamCfg<MB>::kThreads, 2)
gemm_decode_stream_kernel(const __grid_constant__ CUtensorMap x_map, const StreamParams p) {
    static_assert(!FUSEQ || MB == 1, "only a single row is quantized inside the product kernel");
    static_assert(!WIDE || MB == 16, "clusters of 5 to 8 are for the 16-row route");
    extern __shared__ uint8_t smem_raw[];
    using Smem = StreamSmem<MB, WIDE>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr bool kUseMma = StreamCfg<MB>::kUseMma;
    constexpr int kRows = StreamCfg<MB>::kRows;
    constexpr int kStrStages = StreamCfg<MB>::kStages;
    constexpr int kPhases = StreamCfg<MB>::kPhases;
    constexpr int kStrConsumerWarps = StreamCfg<MB>::kConsumerWarps;
    constexpr int kStrThreads = StreamCfg<MB>::kThreads;
    cg::cluster_group cluster = cg::this_cluster();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = k_blocks(p.K);
    const int rank = blockIdx.x, split = gridDim.x;
    const int tile = blockIdx.y;
    const int kb0 = (int)((long long)KB * rank / split), kb1 = (int)((long long)KB * (rank + 1) / split);

    // First meeting of the cluster, arrival only: by the time a CTA writes into another's shared memory
    // (after its k range) every CTA of the cluster has started. The wait comes just before those writes.
    if (split > 1) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    if (threadIdx.x == 0) {
        if constexpr (kRows > 1)     // start the descriptor's fetch now; the first tile load would wait for it
            asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
        for (int s = 0; s < kStrStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(s_u32(&sm.full[s])) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_u32(&sm.empty[s])), "r"(4) : "memory");   // the four quarter warps of the block's phase
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile uint32_t* abort_flag = &sm.abort_flag;
    const uint8_t* wsrc = p.w_packed + (size_t)tile * KB * kBlockBytes;

    // a stage's barrier expects the weight block and the activation codes; the two copies may be issued apart
    // One row is fetched with a plain copy, which must stay inside the row: of a last block that K does
    // not fill, only the codes that exist are copied (a multiple of 32 bytes); the rest of the stage keeps
    // stale bytes, which meet zero weight codes. Tensor-map loads count their whole box.
    auto x_bytes = [&](int kb) -> uint32_t {
        if (FUSEQ) return 0u;                          // the codes are made here, not copied
        return kRows == 1 ? (uint32_t)min(kTileK, p.K - kb * kTileK)
                          : (uint32_t)((kRows == 16 && p.M <= 8 ? 8 : kRows) * kTileK);   // the tensor map's box: 8 rows when M <= 8
    };
    auto issue_w = [&](int kb, int s) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     ::"r"(s_u32(&sm.full[s])), "r"((uint32_t)kBlockBytes + x_bytes(kb)) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(s_u32(sm.w[s])), "l"(wsrc + (size_t)kb * kBlockBytes), "r"((uint32_t)kBlockBytes),
                       "r"(s_u32(&sm.full[s])) : "memory");
    };
    auto issue_x = [&](int kb, int s) {
        if constexpr (FUSEQ) {
        } else if constexpr (kRows == 1) {
            // one row: its 128 codes are contiguous, a plain bulk copy needs no tensor-map fetch
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(s_u32(sm.x[s])), "l"(p.q + (size_t)kb * kTileK), "r"(x_bytes(kb)),
                           "r"(s_u32(&sm.full[s])) : "memory");
        } else {
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                ::"r"(s_u32(sm.x[s])), "l"(&x_map), "r"(kb * kTileK), "r"(0), "r"(s_u32(&sm.full[s])) : "memory");
        }
    };
    // The weights do not depend on the kernel before this one: the first ring of weight blocks is on its
    // way before this grid waits for that kernel (a no-op unless the launch allowed the overlap), and only
    // then are the status word, the codes, the exponent and the offsets touched.
    // Launched with programmatic stream serialization: this grid may have been set up while the kernel
    // before it on the stream still ran. Nothing written before this launch is read, and nothing is written,
    // until that kernel has completed; only behind the call's own quantize kernel (which allows this
    // launch only once everything before it, weight packing included, has completed), or on the caller's
    // promise that nothing in flight writes the weights, the weights are fetched first. With that promise
    // the launch behind this one is also allowed from the start, so that its CTAs take the places of this
    // grid's CTAs as they leave and have their first ring on the way while this grid finishes.
    // The producer is kProdLanes lanes of warp 0 in lockstep, lane l taking the blocks l, l + kProdLanes, ...
    constexpr int kProdLanes = StreamCfg<MB>::kProdLanes;
    const bool producer = warp == 0 && lane < kProdLanes;
    const int ring = min(kStrStages, kb1 - kb0);      // blocks of the first ring
    int issued = 0;
    if (p.early_dependents) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.early_weights) {     // behind this call's own quantize kernel, or the caller has promised stable weights
        if (producer)
            for (int i = lane; i < ring; i += kProdLanes) issue_w(kb0 + i, i);
        issued = ring;
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.clear_status && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) p.ctl->status = 0;   // nothing has given up yet
    [[maybe_unused]] int fused_exp = 0;
    if constexpr (FUSEQ) {
        // ---- the layer scale and this CTA's codes (Eq. 1, Eq. 2 / Eq. 5 with zp = 0; one scale for the layer)
        if (producer)
            for (int i = issued + lane; i < ring; i += kProdLanes) issue_w(kb0 + i, i);   // weights on their way meanwhile
        issued = ring;
        const uint4* xv = reinterpret_cast<const uint4*>(p.x_row + (p.row_idx ? (size_t)p.row_idx[0] * p.K : 0));
        int e = p.clip_shift_or_exp;
        // up to kKeep vectors per thread stay in registers between the two passes (K <= 18432); longer rows
        // are read again (from L2) for the codes
        constexpr int kKeep = 8;
        uint4 keep[kKeep];
        const int n_vec = p.K / 8;
        const bool kept = n_vec <= kKeep * kStrThreads;
        if (p.scale_mode == AQ_SCALE_DYNAMIC || kept) {
            __half2 m2 = __float2half2_rn(0.0f);
            if (kept) {
#pragma unroll
                for (int i = 0; i < kKeep; ++i) {
                    const int v = (int)threadIdx.x + i * kStrThreads;
                    keep[i] = v < n_vec ? __ldg(xv + v) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int i = 0; i < kKeep; ++i) {
                    const __half2* h = reinterpret_cast<const __half2*>(&keep[i]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) m2 = __hmax2(m2, __habs2(h[k]));   // NaN operands are dropped
                }
            } else {
                for (int v = (int)threadIdx.x; v < n_vec; v += kStrThreads) {
                    const uint4 d = __ldg(xv + v);
                    const __half2* h = reinterpret_cast<const __half2*>(&d);
#pragma unroll
                    for (int k = 0; k < 4; ++k) m2 = __hmax2(m2, __habs2(h[k]));
                }
            }
            unsigned int bmax = max((unsigned int)__half_as_ushort(__low2half(m2)), (unsigned int)__half_as_ushort(__high2half(m2)));
            if (bmax > 0x7C00u) bmax = 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) bmax = max(bmax, __shfl_xor_sync(0xFFFFFFFFu, bmax, o));
            if (lane == 0) sm.warp_max[warp] = bmax;
            __syncthreads();
            unsigned int all = 0;
#pragma unroll
            for (int w = 0; w < kStrThreads / 32; ++w) all = max(all, sm.warp_max[w]);
            if (p.scale_mode == AQ_SCALE_DYNAMIC) {
                e = layer_exponent_from_bits(all, p.bits) - p.clip_shift_or_exp;
                if (tile == 0 && rank == 0 && threadIdx.x == 0) p.ctl->absmax_bits = all;
            }
        }
        if (tile == 0 && rank == 0) {
            if (threadIdx.x == 0) { p.ctl->scale_exp = e; p.ctl->status = 0; p.ctl->counter = 0; }
            if (threadIdx.x < 57) p.ctl->split_flags[threadIdx.x] = 0;
        }
        const float lo = -(float)(1 << (p.bits - 1)), hi = (float)((1 << (p.bits - 1)) - 1);
        const int v0 = kb0 * (kTileK / 8), v1 = min(kb1 * (kTileK / 8), p.K / 8);       // 8-element vectors of this k range
        const bool fast = e >= -14 && e <= 14;             // 2^-e is a normal half: codes in half2 arithmetic
        const __half2 inv2 = __float2half2_rn(fast ? __int_as_float((127 - e) << 23) : 1.0f);
        const __half2 lo2 = __float2half2_rn(lo), hi2 = __float2half2_rn(hi);
        auto code8 = [&](const uint4& d, int v) {
            uint2 c;
            if (fast) quantize8_half2(d, inv2, lo2, hi2, c.x, c.y);
            else c = quantize8_fp32(d, e, lo, hi, nullptr);
            reinterpret_cast<uint2*>(sm.xq)[v - v0] = c;
            if (tile == 0) reinterpret_cast<uint2*>(p.q_out)[v] = c;
        };
        if (kept) {
#pragma unroll
            for (int i = 0; i < kKeep; ++i) {
                const int v = (int)threadIdx.x + i * kStrThreads;
                if (v >= v0 && v < v1) code8(keep[i], v);
            }
        } else {
            for (int v = v0 + (int)threadIdx.x; v < v1; v += kStrThreads) code8(__ldg(xv + v), v);
        }
        fused_exp = e;
        __syncthreads();
    }
    if (warp == 0) {
        if (producer) {
            for (int i = lane; i < issued; i += kProdLanes) issue_x(kb0 + i, i);
            for (int kb = kb0 + issued + lane; kb < kb1; kb += kProdLanes) {
                const uint32_t i = (uint32_t)(kb - kb0);
                const int s = (int)(i % kStrStages);
                if (!str_wait(&sm.empty[s], ((i / kStrStages) & 1u) ^ 1u, abort_flag)) break;
                issue_w(kb, s);
                issue_x(kb, s);
            }
        }
    } else {
        const int cw = warp - 1;
        const int quarter = cw & 3, phase = cw >> 2;
        if constexpr (!kUseMma) {
            // A lane takes one 32-k chunk of the block (t = lane / 8) and eight channels per pass (g = lane % 8,
            // four passes cover the warp's 32 channels): per block it reads four 16-byte weight units (chunk t
            // of channels 8i + g; the eight lanes of a quarter warp read eight consecutive units) and the 32
            // activation bytes of its chunk, six 16-byte shared-memory loads where one lane per channel, every
            // lane reading every activation byte, took twelve. The sum over k does not care which lane adds
            // which k; the lanes' partial sums meet once, after the k range.
            const int g = lane & 7, t = lane >> 3;
            int acc[MB][4];
#pragma unroll
            for (int m = 0; m < MB; ++m)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[m][i] = 0;
            for (int kb = kb0 + phase; kb < kb1; kb += kPhases) {       // the warps of a quarter take the k blocks in turn
                const uint32_t it = (uint32_t)(kb - kb0);
                const int s = (int)(it % kStrStages);
                if (!__all_sync(0xFFFFFFFFu, str_wait(&sm.full[s], (it / kStrStages) & 1u, abort_flag) ? 1 : 0)) break;
                uint4 wv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    wv[i] = reinterpret_cast<const uint4*>(sm.w[s])[t * kTileN + quarter * 32 + 8 * i + g];
#pragma unroll
                for (int m = 0; m < MB; ++m) {
                    const uint4* xp = FUSEQ ? reinterpret_cast<const uint4*>(sm.xq + (size_t)(kb - kb0) * kTileK + 32 * t)
                                            : reinterpret_cast<const uint4*>(sm.x[s] + m * kTileK + 32 * t);
                    const uint4 x0 = xp[0], x1 = xp[1];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        // word u of a unit: k 8u..8u+3 of the chunk in its low nibbles, k 8u+4..8u+7 in its high ones
                        const uint32_t w[4] = {wv[i].x, wv[i].y, wv[i].z, wv[i].w};
                        int a = acc[m][i];
                        a = __dp4a((int)((w[0] << 4) & 0xF0F0F0F0u), (int)x0.x, a);      // 16*code
                        a = __dp4a((int)(w[0] & 0xF0F0F0F0u), (int)x0.y, a);
                        a = __dp4a((int)((w[1] << 4) & 0xF0F0F0F0u), (int)x0.z, a);
                        a = __dp4a((int)(w[1] & 0xF0F0F0F0u), (int)x0.w, a);
                        a = __dp4a((int)((w[2] << 4) & 0xF0F0F0F0u), (int)x1.x, a);
                        a = __dp4a((int)(w[2] & 0xF0F0F0F0u), (int)x1.y, a);
                        a = __dp4a((int)((w[3] << 4) & 0xF0F0F0F0u), (int)x1.z, a);
                        a = __dp4a((int)(w[3] & 0xF0F0F0F0u), (int)x1.w, a);
                        acc[m][i] = a;
                    }
                }
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_u32(&sm.empty[s])) : "memory");
            }
            // the four chunks of a channel meet (two exchange steps), then lane (g, t) keeps pass t's channel
            // 8t + g; the warps of a quarter meet in the sum buffer, one after the other (the same thread
            // position owns an element in each of them: the first stores, the others add)
            int mine[MB];
#pragma unroll
            for (int m = 0; m < MB; ++m) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[m][i] += __shfl_xor_sync(0xFFFFFFFFu, acc[m][i], 8);
                    acc[m][i] += __shfl_xor_sync(0xFFFFFFFFu, acc[m][i], 16);
                }
                mine[m] = t == 0 ? acc[m][0] : t == 1 ? acc[m][1] : t == 2 ? acc[m][2] : acc[m][3];
            }
            const int r = quarter * 32 + 8 * t + g;                  // channel inside the tile
#pragma unroll
            for (int ph = 0; ph < kPhases; ++ph) {
                if (ph > 0) asm volatile("bar.sync 1, %0;" ::"n"(kStrConsumerWarps * 32) : "memory");
                if (phase == ph) {
#pragma unroll
                    for (int m = 0; m < MB; ++m) {
                        if (ph == 0) sm.sum[m][r] = mine[m];
                        else sm.sum[m][r] += mine[m];
                    }
                }
            }
        } else {
            // Warp-level int8 MMA, D[16 rows x 8 channels] += A[16 x 32 k] * B[32 k x 8 channels].
            // Fragment owner: g = lane / 4 (row g and g+8 of A and D; channel g of B),
            // t = lane % 4 (k bytes 4t..4t+3 and 16+4t..; D columns 2t, 2t+1).
            // Rows 8..15 are not read when M <= 8. (Splitting a block among the four warps of a phase into channel
            // halves x k halves instead of channel quarters, so that a warp reads half of the activation tile,
            // measured the same within 0.2 us either way.)
            const int g = lane >> 2, t = lane & 3;
            const bool upper = p.M > 8;
            int acc[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[i][c] = 0;
            for (int kb = kb0 + phase; kb < kb1; kb += kPhases) {
                const uint32_t it = (uint32_t)(kb - kb0);
                const int s = (int)(it % kStrStages);
                if (!__all_sync(0xFFFFFFFFu, str_wait(&sm.full[s], (it / kStrStages) & 1u, abort_flag) ? 1 : 0)) break;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // The sum over k does not depend on which k sits in which slot of the instruction, as long
                    // as both operands agree: lane t feeds its slots "k 4t.." and "k 16+4t.." with the k range
                    // 8t..8t+3 and 8t+4..8t+7 of this 32-k chunk, i.e. with the two nibble planes of ONE packed
                    // word and eight consecutive activation bytes (one 8-byte load per row).
                    // activation rows: 128 bytes, 16-byte chunks XOR-swizzled by row % 8
                    const int x_off = (((2 * j + (t >> 1)) ^ g) << 4) + 8 * (t & 1);
                    const uint2 xa = *reinterpret_cast<const uint2*>(sm.x[s] + g * kTileK + x_off);
                    uint2 xb = make_uint2(0u, 0u);
                    if (upper) xb = *reinterpret_cast<const uint2*>(sm.x[s] + (g + 8) * kTileK + x_off);
                    const uint32_t a0 = xa.x, a1 = xb.x, a2 = xa.y, a3 = xb.y;
                    // Weight fragments of the four channel passes in one instruction: the 32 units (16 bytes each)
                    // of this chunk and channel quarter are four 8 x 8 matrices of 16-bit elements, one per pass;
                    // lane l gives the address of unit l, and lane (g, t) receives word t of channel 8i + g for
                    // i = 0..3, which holds k 8t..8t+3 in its low nibbles and k 8t+4..8t+7 in its high nibbles.
                    uint32_t pw[4];
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(pw[0]), "=r"(pw[1]), "=r"(pw[2]), "=r"(pw[3])
                                 : "r"(s_u32(sm.w[s] + (size_t)(j * kTileN + quarter * 32 + lane) * 16)) : "memory");
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t b0 = (pw[i] << 4) & 0xF0F0F0F0u;
                        const uint32_t b1 = pw[i] & 0xF0F0F0F0u;
                        asm volatile(
                            "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
                            "{%8, %9}, {%0, %1, %2, %3};"
                            : "+r"(acc[i][0]), "+r"(acc[i][1]), "+r"(acc[i][2]), "+r"(acc[i][3])
                            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
                    }
                }
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_u32(&sm.empty[s])) : "memory");
            }
            // D fragment: acc[i][0..1] = row g, channels 8i+2t, +1; acc[i][2..3] = row g+8.
            // The warps of a quarter meet in the sum buffer, one after the other (the same thread position
            // owns an element in each of them: the first stores, the others add).
#pragma unroll
            for (int ph = 0; ph < kPhases; ++ph) {
                if (ph > 0) asm volatile("bar.sync 1, %0;" ::"n"(kStrConsumerWarps * 32) : "memory");
                if (phase == ph) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            int& dst = sm.sum[g + 8 * (c >> 1)][quarter * 32 + 8 * i + 2 * t + (c & 1)];
                            if (ph == 0) dst = acc[i][c];
                            else dst += acc[i][c];
                        }
                }
            }
        }
    }
    // Every CTA of the cluster now holds the tile's sums over its own k range, and CTA `rank` finishes the
    // tile's channel slice `rank`: every CTA writes its sums of the other slices into
    // their owners' shared memory (slot = sender), the cluster meets once, and every CTA adds what it received
    // to its own sums (integer addition is exact in any order), scales and writes its outputs. After the
    // meeting nobody touches another CTA's memory, so a CTA may leave as soon as it is done. (Reading the
    // other CTAs' sums over distributed shared memory instead, with a second meeting before anybody leaves,
    // measured 0.1-0.5 us slower at every row count.)
    // The scale is fetched before the cluster meets so that its latency overlaps the wait.
    // This CTA's k range is done: a launch behind this one that allows it may be scheduled and set up now
    // (it reads and writes nothing before this grid has completed).
    if (!p.early_dependents) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Channel slices: 128 / split channels each for split 1, 2, 4 (divisions are shifts). Clusters of 5 to 8
    // (16-row route on long k ranges) cut the tile's 32 groups of four channels into `split` nearly equal
    // runs, slice r = groups [32 r / split, 32 (r + 1) / split): at most 28 channels, handled by the first
    // lanes of 32-thread rows.
    constexpr bool wide = WIDE;                                // this instantiation is launched with clusters of 5 to 8
    const int cw = wide ? 32 : kTileN / split;                // slot width in the receive buffer
    const int cw_log = wide ? 5 : 7 - (31 - __clz(split));
    const int g_first = (32 * rank) / split, g_count = (32 * (rank + 1)) / split - g_first;   // this CTA's groups (wide)
    const int ft = (int)threadIdx.x - 32;                     // the consumer threads finish (a multiple of 128 = 4 cw at most)
    const int rc = ft & (cw - 1);                             // channel inside the slice (only used when ft >= 0)
    const int out_r = wide ? 4 * g_first + rc : rank * cw + rc;
    const int out_n = tile * kTileN + out_r;
    const bool mine = ft >= 0 && out_n < p.N && (!wide || rc < 4 * g_count);
    float sc = 0.0f, off = 0.0f;
    if (mine) {
        const float pe = __int_as_float((127 + (FUSEQ ? fused_exp : *p.scale_exp)) << 23);
        sc = __half2float(p.w_scales[out_n]) * pe;
        if (p.chan_offset) off = p.chan_offset[out_n] * pe;
    }
    const int rows = p.M < kRows ? p.M : kRows;
    if (split > 1) {
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");     // everybody has started (arrival at the top)
        __syncthreads();                                      // this CTA's sums are complete
        if (ft >= 0) {
            // four consecutive channels at a time (16-byte remote stores) go to the CTA that owns them
            for (int e = ft; e < rows * (kTileN / 4); e += kStrConsumerWarps * 32) {
                const int m = e >> 5, g4 = e & 31, ch = 4 * g4;
                const int owner = wide ? (((g4 + 1) * split + 31) >> 5) - 1 : ch >> cw_log;
                const int at = wide ? ch - 4 * ((32 * owner) / split) : ch & (cw - 1);   // place inside the owner's slice
                if (owner != rank)
                    *reinterpret_cast<int4*>(cluster.map_shared_rank(&sm.recv[0][0], owner) + m * Smem::kRecvStride + rank * cw + at) =
                        *reinterpret_cast<const int4*>(&sm.sum[m][ch]);
            }
        }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
    if (mine) {
        // All shared-memory reads of this thread's outputs are issued before the first is used and without
        // branches around them (rows that do not exist read the last row of the buffer and are dropped):
        // taken one after the other, each behind its own test, they were the longest part of the finish at
        // 16 rows.
        constexpr int kIt = (kRows + kPhases - 1) / kPhases;      // a pass of the consumer threads covers at least kPhases rows
        const int stride = (kStrConsumerWarps * 32) >> cw_log, m0 = ft >> cw_log;
        int av[kIt];
#pragma unroll
        for (int i = 0; i < kIt; ++i) av[i] = i * stride < kRows ? sm.sum[min(m0 + i * stride, kRows - 1)][out_r] : 0;
#pragma unroll
        for (int k = 1; k < (WIDE ? 8 : 4); ++k) {
            if (k < split) {
                int c = rank + k;                                             // the k-th other CTA's slot
                if (c >= split) c -= split;
                const int col = c * cw + rc;
#pragma unroll
                for (int i = 0; i < kIt; ++i)
                    if (i * stride < kRows) av[i] += sm.recv[min(m0 + i * stride, kRows - 1)][col];   // the same test in every thread
            }
        }
        if (!p.acc_dump && !p.q_next) {
#pragma unroll
            for (int i = 0; i < kIt; ++i) {
                const int m = m0 + i * stride;
                const __half hv = __float2half_rn(fmaf((float)(av[i] >> 4), sc, off));     // sums carry a factor 16
                if (m < rows) p.y[(size_t)m * p.N + out_n] = hv;
            }
        } else {
#pragma unroll
            for (int i = 0; i < kIt; ++i) {
                const int m = m0 + i * stride;
                if (m < rows) {
                    const int a = av[i] >> 4;
                    if (p.acc_dump) p.acc_dump[(size_t)m * p.N + out_n] = a;
                    const __half hv = __float2half_rn(fmaf((float)a, sc, off));
                    // (a warp's lanes hold consecutive channels and run this loop together: slices of 32 and
                    // more channels; clusters of 5 to 8 are not used with chained outputs)
                    if (p.q_next)
                        store_next_code(p.q_next, (size_t)m * p.N + out_n, next_code(hv, p.next_inv, p.next_lo, p.next_hi),
                                        p.next_packed, true, lane);
                    else p.y[(size_t)m * p.N + out_n] = hv;
                }
            }
        }
    }
    if (sm.abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);          // let copies in flight land
        if (threadIdx.x == 0) atomicOr(&p.ctl->status, 1u);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// k ranges per tile by the usual rule: 1, 2 or 4, as many as keep all CTAs resident at once (two per SM) with at
// least two k blocks per CTA (wide_split_for may raise a 4 to 5..8 for the 16-row route)
inline int decode_split(int tiles, int KB, int sm_count) {
    int split = 1;
    while (split < 4 && tiles * split * 2 <= 2 * sm_count && KB / (split * 2) >= 2) split *= 2;
    return split;
}

template <int MB, bool FUSEQ = false, bool WIDE = false>
cudaError_t launch_stream(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream, int wide_split = 0) {
    using Smem = StreamSmem<MB, WIDE>;
    const size_t smem_bytes = sizeof(Smem) + 1024;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(gemm_decode_stream_kernel<MB, FUSEQ, WIDE>, dev.device, smem_bytes); e != cudaSuccess)
        return e;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
    const cuuint64_t strides[1] = {(cuuint64_t)a.K};
    // 16-row route: rows 8..15 are neither copied nor read when M <= 8
    const cuuint32_t box[2] = {128u, (cuuint32_t)(StreamCfg<MB>::kRows == 16 && a.M <= 8 ? 8 : StreamCfg<MB>::kRows)};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(dev.encode_tiled)(
        &map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(a.q), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE,
        StreamCfg<MB>::kUseMma ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
        CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    StreamParams p;
    p.M = a.M; p.K = a.K; p.N = a.N; p.Npad = round_up(a.N, kTileN);
    p.q = a.q;
    p.clear_status = a.after_quantize ? 0 : 1;
    p.next_packed = a.next_packed ? 1 : 0;
    p.w_packed = a.w_packed; p.w_scales = a.w_scales; p.scale_exp = a.scale_exp;
    p.y = a.y; p.acc_dump = a.acc_dump; p.ctl = a.ctl; p.chan_offset = a.chan_offset;
    p.q_next = a.q_next;
    p.next_inv = ldexpf(1.0f, -a.next_exp);
    p.next_lo = -(float)(1 << (a.next_bits - 1));
    p.next_hi = (float)((1 << (a.next_bits - 1)) - 1);
    p.x_row = a.fuse_x; p.row_idx = a.fuse_row_idx; p.q_out = const_cast<int8_t*>(a.q);
    p.bits = a.fuse_bits; p.scale_mode = a.fuse_scale_mode; p.clip_shift_or_exp = a.fuse_clip_shift_or_exp;
    if (FUSEQ) p.clear_status = 1;       // no quantize kernel of this call runs ahead
    // Weights ahead of the wait: behind the call's own quantize kernel (which allows this launch only once
    // everything before it has completed), or on the caller's promise that nothing in flight writes them.
    p.early_weights = (!p.clear_status || a.weights_stable) ? 1 : 0;
    p.early_dependents = a.weights_stable ? 1 : 0;
    const int tiles = p.Npad / kTileN, KB = k_blocks(a.K);
    const int split = WIDE ? wide_split : decode_split(tiles, KB, dev.sm_count);
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(StreamCfg<MB>::kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(split, tiles, 1);
    attr[0].val.clusterDim.x = split;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;       // the kernel reads and writes nothing before the kernel ahead of it has completed
    return cudaLaunchKernelEx(&cfg, gemm_decode_stream_kernel<MB, FUSEQ, WIDE>, map, p);
}

// 16-row route: its consumers, not the memory, set a CTA's pace, so more CTAs per tile pay as long as each
// keeps five k blocks and all clusters still run at once (a GPC holds only so many clusters of a size: the
// occupancy query says how many the device does). Measured on the 13B shapes with N = 5120 (clusters of 7):
// K = 13824 12.5 / 13.2 -> 9.8 / 10.4 us at M = 4 / 16, K = 5120 6.9 / 7.3 -> 6.0 / 6.5 us; a single row
// loses with clusters of 8 (N = 4096, K = 5120: 5.1 -> 6.2 us). Chained outputs keep slices of at least 32
// channels. Returns the cluster size (5 to 8), or 0 for the usual 1, 2 or 4.
int wide_split_for(const GemmArgs& a, const DeviceInfo& dev) {
    const int tiles = round_up(a.N, kTileN) / kTileN, KB = k_blocks(a.K);
    if (a.q_next || decode_split(tiles, KB, dev.sm_count) != 4) return 0;
    static std::atomic<int> fits[kMaxDevices][9];               // clusters of s that run at once, + 1 (0: not asked yet)
    int s = (2 * dev.sm_count) / tiles;
    if (s > 8) s = 8;
    for (; s > 4; --s) {
        if (KB / s < 5) continue;
        int known = fits[dev.device][s].load(std::memory_order_relaxed);
        if (known == 0) {
            using Smem = StreamSmem<16, true>;
            const size_t smem_bytes = sizeof(Smem) + 1024;
            static SmemOptIn opt_in;
            int n = 0;
            if (opt_in.ensure(gemm_decode_stream_kernel<16, false, true>, dev.device, smem_bytes) == cudaSuccess) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(s, tiles, 1);
                cfg.blockDim = dim3(StreamCfg<16>::kThreads);
                cfg.dynamicSmemBytes = smem_bytes;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = s;
                attr[0].val.clusterDim.y = 1;
                attr[0].val.clusterDim.z = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 1;
                if (cudaOccupancyMaxActiveClusters(&n, gemm_decode_stream_kernel<16, false, true>, &cfg) != cudaSuccess) {
                    (void)cudaGetLastError();
                    n = 0;
                }
            }
            known = n + 1;
            fits[dev.device][s].store(known, std::memory_order_relaxed);
        }
        if (known - 1 >= tiles) return s;
    }
    return 0;
}

template <int MB>
cudaError_t launch_mb(const GemmArgs& a, cudaStream_t stream) {
    const int Npad = round_up(a.N, kTileN);
    dim3 grid(Npad / 32, (a.M + MB - 1) / MB);
    if (a.group)
        gemm_decode_kernel<MB, true><<<grid, kDecThreads, 0, stream>>>(
            a.q, a.M, a.K, a.N, Npad, a.w_packed, a.w_scales, a.scale_exp, a.y, a.acc_dump, a.ctl, a.chan_offset,
            a.q_next, ldexpf(1.0f, -a.next_exp), -(float)(1 << (a.next_bits - 1)), (float)((1 << (a.next_bits - 1)) - 1),
            a.after_quantize ? 0 : 1, a.next_packed ? 1 : 0);
    else
        gemm_decode_kernel<MB, false><<<grid, kDecThreads, 0, stream>>>(
            a.q, a.M, a.K, a.N, Npad, a.w_packed, a.w_scales, a.scale_exp, a.y, a.acc_dump, a.ctl, a.chan_offset,
            a.q_next, ldexpf(1.0f, -a.next_exp), -(float)(1 << (a.next_bits - 1)), (float)((1 << (a.next_bits - 1)) - 1),
            a.after_quantize ? 0 : 1, a.next_packed ? 1 : 0);
    return cudaGetLastError();
}

}  // namespace

// One row, one scale per channel, and a k range per CTA that fits the kernel's code buffer: the product
// kernel can quantize the row itself (one launch for the layer).
bool decode_can_fuse_quantize(int M, int K, int N, int group, int sm_count) {
    if (M != 1 || group) return false;
    const int tiles = round_up(N, kTileN) / kTileN, KB = k_blocks(K);
    const int split = decode_split(tiles, KB, sm_count);
    return (KB + split - 1) / split + 1 <= kFuseMaxBlocks;
}

cudaError_t launch_gemm_decode(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    if (!a.group && a.M <= 16) {
        // one row: dp4a; 2..16 rows: the warp MMA on a 16-row tile (fewer instructions per weight
        // chunk than dp4a from two rows on; measured faster at M = 4: 7.5 / 11.1 / 13.3 us against
        // 8.1 / 12.8 / 15.2 us on the three 13B shapes)
        if (a.M <= 1 && a.fuse_x) return launch_stream<1, true>(a, dev, stream);
        if (a.M <= 1) return launch_stream<1>(a, dev, stream);
        if (const int ws = wide_split_for(a, dev)) return launch_stream<16, false, true>(a, dev, stream, ws);
        return launch_stream<16>(a, dev, stream);
    }
    if (a.M <= 1) return launch_mb<1>(a, stream);
    if (a.M <= 2) return launch_mb<2>(a, stream);
    if (a.M <= 4) return launch_mb<4>(a, stream);
    if (a.M <= 8) return launch_mb<8>(a, stream);
    return launch_mb<16>(a, stream);
}

}  // namespace aq

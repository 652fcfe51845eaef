// Integer product with one scale per output channel (Sec. 4.4) on tiles of 256 channels x 128 or 192 tokens.
//
// The per-channel kernel of aq_gemm_tensor.cu moves 40 KB from L2 per 128-k block and SM (a 256-token
// activation tile and one packed 128-channel weight block) and runs within 20 % of what the L2 -> SM path
// delivers for that pattern. Here a CTA's tile covers TWO adjacent 128-channel blocks that share one
// activation tile of 128 or 192 tokens: 32 KB per k block for the products of 40 KB there, or 40 KB for one
// and a half times as many, so the same path feeds a fifth to a half more work. The two channel halves are
// two accumulators in tensor memory, each fed by its own MMA-issuing thread from its own weight slices, which
// its own group of four unpack warps writes; the activation tile in shared memory is the B operand of both.
// Each half has its own pair of accumulator barriers: the epilogue takes the halves one after the other.
// Roles: warp 0 = TMA producer of the activation tiles, warp 2 = of the two weight blocks, warps 1 and 3 =
// MMA issuers (half 0 / half 1), warps 4-7 and 8-11 = unpack (half 0 / half 1), warps 12-19 = epilogue.
// Needs an even number of 128-channel blocks; other shapes take the kernel of aq_gemm_tensor.cu.
#include <cuda.h>

#include "aq_common.cuh"
#include "aq_tc.cuh"

namespace aq {

namespace {

constexpr int kWThreads = 20 * 32;
constexpr int kWFirstUnpack = 4, kWFirstEpi = 12, kWEpiWarps = 8;
constexpr int kWRegsControl = 40, kWRegsUnpack = 48, kWRegsEpi = 168;     // of the 96 x 640 the launch allocates
static_assert(128 * kWRegsControl + 256 * kWRegsUnpack + 256 * kWRegsEpi <= kWThreads * 96,
              "register plan exceeds the launch allocation");
constexpr int kWStageRows = 32;           // tokens per TMA store of an epilogue warp
template <int BM>
struct WCfg {
    static constexpr int kStages = BM == 128 ? 6 : 5;          // shared-memory ring: activation tile + two packed weight blocks per stage
    static constexpr int kSlices = (512 - 2 * BM) / 32;        // weight slices in tensor memory: (k block, half) pairs: 8 or 4
    static constexpr int kAccCols = 2 * BM;                    // two accumulators (one per channel half)
    static constexpr int kCols = BM / 2;                       // token columns of one epilogue warp (per half)
    static_assert(kCols % kWStageRows == 0 && kCols <= 96, "epilogue register plan");
};

template <int BM>
struct WSmem {
    static constexpr int kStages = WCfg<BM>::kStages;
    alignas(1024) uint8_t x[kStages][BM * 128];                // activation tiles, 128-byte swizzled rows
    alignas(128) uint8_t w[kStages][2][kBlockBytes];           // the two packed weight blocks of a k block
    alignas(128) __half ystage[kWEpiWarps][kWStageRows][32];
    alignas(8) uint64_t tma_full[kStages];                     // both producers' bytes landed -> unpack warps
    uint64_t smem_empty[kStages];                              // both halves' MMAs done -> TMA producers
    uint64_t a_full[8];                                        // a half's unpack warps stored the slice -> its MMA issuer
    uint64_t a_empty[8];                                       // MMA done with the slice -> unpack warps
    uint64_t acc_full[2];                                      // a half's last MMAs of the tile done -> epilogue
    uint64_t acc_empty[2];                                     // epilogue has the half's sums in registers -> its issuer
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
};

struct WParams {
    int M, K, N, Npad, KB;
    int n_tiles_m, n_tiles;        // token tiles; tiles (token tile x channel pair)
    const uint8_t* w_packed;
    const __half* w_scales;
    const int32_t* scale_exp;
    __half* y;
    int32_t* acc_dump;
    Control* ctl;
    const float* chan_offset;
    int8_t* q_next;
    float next_inv, next_lo, next_hi;
    int next_packed;
    int y_tma;
};

__device__ __forceinline__ int w_chain_code(__half hv, float inv, float lo, float hi) {
    const float t = __half2float(hv) * inv;                 // exact: inv is a power of two
    if (t != t) return 0;
    return (int)fminf(fmaxf(rintf(t), lo), hi);
}
__device__ __forceinline__ void w_stage_code(__half* stage, int c, int lane, int code, int packed) {
    if (packed) {
        const int hi = __shfl_down_sync(0xFFFFFFFFu, code, 1);
        if (!(lane & 1)) reinterpret_cast<uint8_t*>(stage)[c * 16 + (lane >> 1)] = (uint8_t)((code & 0xF) | (hi << 4));
    } else {
        reinterpret_cast<int8_t*>(stage)[c * 32 + lane] = (int8_t)code;
    }
}

// OFFSET: add the per-channel term of the zero-point variant. CHAIN: write the next layer's codes instead
// of fp16 outputs.
template <int BM, bool OFFSET, bool CHAIN>
__global__ void __launch_bounds__(kWThreads, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap y_map, const WParams p) {
    extern __shared__ uint8_t smem_raw[];
    using Smem = WSmem<BM>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kWBM = BM, kWStages = WCfg<BM>::kStages, kWSlices = WCfg<BM>::kSlices, kWAccCols = WCfg<BM>::kAccCols;
    constexpr int kCols = WCfg<BM>::kCols;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = p.KB;
    const int my_tiles = p.n_tiles > (int)blockIdx.x ? (p.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const uint32_t total_iters = (uint32_t)my_tiles * (uint32_t)KB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kWStages; ++s) {
            mbar_init(&sm.tma_full[s], 2);
            mbar_init(&sm.smem_empty[s], 2);
        }
        for (int i = 0; i < kWSlices; ++i) {
            mbar_init(&sm.a_full[i], 4);
            mbar_init(&sm.a_empty[i], 1);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(&sm.acc_full[h], 1);
            mbar_init(&sm.acc_empty[h], kWEpiWarps);
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sm.tmem_base)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tmem_acc = tmem;                 // half h at column h * BM
    const uint32_t tmem_a = tmem + kWAccCols;       // then the slices of 32 columns
    volatile uint32_t* abort_flag = &sm.abort_flag;

    if (warp < kWFirstUnpack) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kWRegsControl));
        if (warp == 0 || warp == 2) {
            // ------------- TMA producers
            if (lane == 0) {
                // behind the call's own quantize kernel (programmatic stream serialization) the codes are
                // touched only after that grid has completed; the weight producer does not wait
                if (warp == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
                uint32_t it = 0;
                for (int tl = 0; tl < my_tiles; ++tl) {
                    const int tile = (int)(blockIdx.x + tl * gridDim.x);
                    const int mt = tile % p.n_tiles_m, np = tile / p.n_tiles_m;
                    const uint8_t* wsrc0 = p.w_packed + (size_t)(2 * np) * KB * kBlockBytes;
                    const uint8_t* wsrc1 = wsrc0 + (size_t)KB * kBlockBytes;
                    for (int kb = 0; kb < KB; ++kb, ++it) {
                        const int s = (int)(it % kWStages);
                        if (!mbar_wait(&sm.smem_empty[s], ((it / kWStages) & 1u) ^ 1u, abort_flag, 1u)) goto role_done;
                        if (warp == 0) {
                            mbar_arrive_expect_tx(&sm.tma_full[s], kWBM * 128);
                            tma_load_2d(sm.x[s], &x_map, kb * kTileK, mt * kWBM, &sm.tma_full[s]);
                        } else {
                            mbar_arrive_expect_tx(&sm.tma_full[s], 2 * kBlockBytes);
                            tma_load_1d(sm.w[s][0], wsrc0 + (size_t)kb * kBlockBytes, kBlockBytes, &sm.tma_full[s]);
                            tma_load_1d(sm.w[s][1], wsrc1 + (size_t)kb * kBlockBytes, kBlockBytes, &sm.tma_full[s]);
                        }
                    }
                }
            }
        } else {
            // ------------- MMA issuers: warp 1 = channel half 0, warp 3 = half 1
            const int h = warp >> 1;
            if (lane == 0) {
                constexpr uint32_t idesc = idesc_i8(128, kWBM);
                uint32_t it = 0;
                for (int tl = 0; tl < my_tiles; ++tl) {
                    if (!mbar_wait(&sm.acc_empty[h], ((uint32_t)tl & 1u) ^ 1u, abort_flag, 4u)) goto role_done;
                    for (int kb = 0; kb < KB; ++kb, ++it) {
                        const int s = (int)(it % kWStages);
                        const uint32_t u = it * 2u + (uint32_t)h;            // this half's slice of the block
                        const int ai = (int)(u % kWSlices);
                        // the unpack warps publish a slice only after the stage's TMA bytes (activation tile
                        // included) have landed, so this one wait covers both operands
                        if (!mbar_wait(&sm.a_full[ai], (u / kWSlices) & 1u, abort_flag, 5u)) goto role_done;
                        tc_fence_after();
                        const uint32_t d_addr = tmem_acc + (uint32_t)(h * kWBM);
                        const uint32_t a_addr = tmem_a + (uint32_t)(ai * kAColsPerStage);
                        const uint64_t bdesc = smem_desc_sw128(smem_u32(sm.x[s]));
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            tc_mma_i8_ts(d_addr, a_addr + 8 * j, bdesc + (uint64_t)(2 * j), idesc, (kb == 0 && j == 0) ? 0u : 1u);
                        tc_commit(&sm.a_empty[ai]);
                        tc_commit(&sm.smem_empty[s]);
                    }
                    tc_commit(&sm.acc_full[h]);
                }
            }
        }
    } else if (warp < kWFirstEpi) {
        // --------------------------------------------------- weight unpack -> tensor memory (one group per half)
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kWRegsUnpack));
        const int quarter = warp & 3;
        const int h = (warp - kWFirstUnpack) >> 2;
        const int r = quarter * 32 + lane;            // row inside the half's 128-channel block = TMEM lane
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        int pending = -1;                             // slice whose stores have been issued but not published
        for (uint32_t it = 0; it < total_iters; ++it) {
            const int s = (int)(it % kWStages);
            const uint32_t u = it * 2u + (uint32_t)h;
            const int ai = (int)(u % kWSlices);
            if (!mbar_wait_warp(&sm.tma_full[s], (it / kWStages) & 1u, abort_flag, 6u)) goto role_done;
            const uint4* src = reinterpret_cast<const uint4*>(sm.w[s][h]) + r;
            uint4 d[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) d[j] = src[j * kTileN];
            if (pending >= 0) {                       // the previous stores had the loads above to finish
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.a_full[pending]);
            }
            if (!mbar_wait_warp(&sm.a_empty[ai], ((u / kWSlices) & 1u) ^ 1u, abort_flag, 7u)) goto role_done;
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t w[4] = {d[j].x, d[j].y, d[j].z, d[j].w};
                uint32_t v[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[2 * i] = (w[i] << 4) & 0xF0F0F0F0u;           // 16*code for k0..k0+3
                    v[2 * i + 1] = w[i] & 0xF0F0F0F0u;              // 16*code for k0+4..k0+7
                }
                tc_st8(tmem_a + lane_addr + (uint32_t)(ai * kAColsPerStage + 8 * j), v);
            }
            pending = ai;
        }
        if (pending >= 0) {
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.a_full[pending]);
        }
    } else {
        // ----------------------------------------------------------------------- epilogue
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kWRegsEpi));
        const int ew = warp - kWFirstEpi;
        const int quarter = warp & 3;
        const int chalf = ew >> 2;                    // which half of the tile's token columns
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int col0 = chalf * kCols;
        asm volatile("griddepcontrol.wait;" ::: "memory");               // see the activation producer
        const float pe = __int_as_float((127 + *p.scale_exp) << 23);     // 2^e
        __half* stage = &sm.ystage[ew][0][0];
        for (int tl = 0; tl < my_tiles; ++tl) {
            const int tile = (int)(blockIdx.x + tl * gridDim.x);
            const int mt = tile % p.n_tiles_m, np = tile / p.n_tiles_m;
            const int m_base = mt * kWBM + col0;
            float sc[2], off_pe[2];
            bool n_ok[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int n = (2 * np + h) * kTileN + r;
                n_ok[h] = n < p.N;
                sc[h] = __half2float(p.w_scales[n]) * 0.0625f * pe;      // sums carry a factor 16 (n < Npad: the scale array is padded)
                off_pe[h] = (OFFSET && n_ok[h]) ? p.chan_offset[n] * pe : 0.0f;
            }
            // One half after the other: the half's sums (this warp's columns) go to registers and its
            // accumulator returns to its issuer at once, so that conversion and stores overlap the next tile's MMAs.
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (!mbar_wait_warp(&sm.acc_full[h], (uint32_t)tl & 1u, abort_flag, 8u)) goto role_done;
                tc_fence_after();
                uint32_t v[kCols];
#pragma unroll
                for (int c0 = 0; c0 < kCols; c0 += 32)
                    tc_ld32(tmem_acc + lane_addr + (uint32_t)(h * kWBM + col0 + c0), *reinterpret_cast<uint32_t(*)[32]>(&v[c0]));
                tc_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.acc_empty[h]);
                const int n = (2 * np + h) * kTileN + r;
                const int n0 = (2 * np + h) * kTileN + quarter * 32;
                if (p.y_tma) {
#pragma unroll
                    for (int r0 = 0; r0 < kCols; r0 += kWStageRows) {
                        if (lane == 0) tma_store_wait_read();     // the previous store has read the staging rows
                        __syncwarp();
#pragma unroll
                        for (int c = 0; c < kWStageRows; ++c) {
                            const __half hv = __float2half_rn(OFFSET ? fmaf((float)(int)v[r0 + c], sc[h], off_pe[h])
                                                                     : (float)(int)v[r0 + c] * sc[h]);
                            if constexpr (CHAIN)
                                w_stage_code(stage, c, lane, w_chain_code(hv, p.next_inv, p.next_lo, p.next_hi), p.next_packed);
                            else
                                stage[c * 32 + lane] = hv;
                        }
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0 && n0 < p.N && m_base + r0 < p.M)
                            tma_store_2d(&y_map, stage, (CHAIN && p.next_packed) ? n0 >> 1 : n0, m_base + r0);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < kCols; ++c) {
                        const int m = m_base + c;
                        if (n_ok[h] && m < p.M) {
                            const __half hv = __float2half_rn(OFFSET ? fmaf((float)(int)v[c], sc[h], off_pe[h])
                                                                     : (float)(int)v[c] * sc[h]);
                            if constexpr (CHAIN)
                                p.q_next[(size_t)m * p.N + n] = (int8_t)w_chain_code(hv, p.next_inv, p.next_lo, p.next_hi);
                            else
                                p.y[(size_t)m * p.N + n] = hv;
                        }
                    }
                }
                if (p.acc_dump) {
#pragma unroll
                    for (int c = 0; c < kCols; ++c) {
                        const int m = m_base + c;
                        if (n_ok[h] && m < p.M) p.acc_dump[(size_t)m * p.N + n] = (int)v[c] >> 4;
                    }
                }
            }
        }
    }

role_done:
    if (warp >= kWFirstEpi && lane == 0) tma_store_wait_read();   // staging rows live until read
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (sm.abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);          // let copies in flight land
        if (threadIdx.x == 0) atomicCAS(&p.ctl->status, 0u, sm.abort_flag);
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

typedef CUresult (*WEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <int BM, bool OFFSET, bool CHAIN>
cudaError_t launch_wide_t(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    constexpr int kWBM = BM;
    const size_t smem_bytes = sizeof(WSmem<BM>) + 1024;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(gemm_wide_kernel<BM, OFFSET, CHAIN>, dev.device, smem_bytes); e != cudaSuccess)
        return e;
    WEncodeTiledFn enc = reinterpret_cast<WEncodeTiledFn>(dev.encode_tiled);
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
    const cuuint64_t strides[1] = {(cuuint64_t)a.K};
    const cuuint32_t box[2] = {128u, (cuuint32_t)kWBM};
    const cuuint32_t estr[2] = {1u, 1u};
    if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(a.q), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    CUtensorMap ymap = map;   // placeholder when the store path is off
    int y_tma = 0;
    if (CHAIN) {
        if (a.next_packed && (a.N % 32 != 0 || (reinterpret_cast<uintptr_t>(a.q_next) & 15u) != 0))
            return cudaErrorInvalidValue;                    // packed codes only leave through the TMA store
        if (a.N % 16 == 0 && (reinterpret_cast<uintptr_t>(a.q_next) & 15u) == 0) {
            const cuuint64_t row_bytes = a.next_packed ? (cuuint64_t)a.N / 2 : (cuuint64_t)a.N;
            const cuuint64_t ydims[2] = {row_bytes, (cuuint64_t)a.M};
            const cuuint64_t ystrides[1] = {row_bytes};
            const cuuint32_t ybox[2] = {a.next_packed ? 16u : 32u, (cuuint32_t)kWStageRows};
            if (enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, a.q_next, ydims, ystrides, ybox, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
            y_tma = 1;
        }
    } else if (a.N % 8 == 0 && (reinterpret_cast<uintptr_t>(a.y) & 15u) == 0) {
        const cuuint64_t ydims[2] = {(cuuint64_t)a.N, (cuuint64_t)a.M};
        const cuuint64_t ystrides[1] = {(cuuint64_t)a.N * 2};
        const cuuint32_t ybox[2] = {32u, (cuuint32_t)kWStageRows};
        if (enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, a.y, ydims, ystrides, ybox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        y_tma = 1;
    }
    WParams p;
    p.M = a.M; p.K = a.K; p.N = a.N; p.Npad = round_up(a.N, kTileN); p.KB = k_blocks(a.K);
    p.n_tiles_m = (a.M + kWBM - 1) / kWBM;
    p.n_tiles = p.n_tiles_m * (p.Npad / (2 * kTileN));
    p.w_packed = a.w_packed; p.w_scales = a.w_scales; p.scale_exp = a.scale_exp;
    p.y = a.y; p.acc_dump = a.acc_dump; p.ctl = a.ctl; p.chan_offset = a.chan_offset;
    p.q_next = a.q_next;
    p.next_inv = ldexpf(1.0f, -a.next_exp);
    p.next_lo = -(float)(1 << (a.next_bits - 1));
    p.next_hi = (float)((1 << (a.next_bits - 1)) - 1);
    p.next_packed = a.next_packed ? 1 : 0;
    p.y_tma = y_tma;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_tiles < dev.sm_count ? p.n_tiles : dev.sm_count);
    cfg.blockDim = dim3(kWThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.after_quantize ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, gemm_wide_kernel<BM, OFFSET, CHAIN>, map, ymap, p);
}

}  // namespace

bool gemm_wide_applies(const GemmArgs& a) {
    return !a.group && a.M > 128 && (round_up(a.N, kTileN) / kTileN) % 2 == 0;
}

namespace {
template <int BM>
cudaError_t launch_wide_bm(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    if (a.q_next) {
        if (a.chan_offset) return cudaErrorInvalidValue;       // the two variants are not combined
        return launch_wide_t<BM, false, true>(a, dev, stream);
    }
    if (a.chan_offset) return launch_wide_t<BM, true, false>(a, dev, stream);
    return launch_wide_t<BM, false, false>(a, dev, stream);
}
}  // namespace

// Token tile: rounds of tiles over the SMs x k blocks x the time of a k block, which the L2 -> SM path sets
// (about 36 bytes per clock and SM measured in this kernel: 32 KB per k block on 128-token tiles, 40 KB on
// 192-token tiles) unless the tensor pipe's 512 / 768 cycles are longer.
int wide_token_tile(int M, int N, int sm_count) {
    const long pairs = round_up(N, kTileN) / (2 * kTileN);
    auto cost = [&](int bm, long unit_cycles) {
        const long tiles = (long)((M + bm - 1) / bm) * pairs;
        return ((tiles + sm_count - 1) / sm_count) * unit_cycles;
    };
    return cost(192, 1138) < cost(128, 910) ? 192 : 128;
}

cudaError_t launch_gemm_wide(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    return wide_token_tile(a.M, a.N, dev.sm_count) == 192 ? launch_wide_bm<192>(a, dev, stream)
                                                          : launch_wide_bm<128>(a, dev, stream);
}

}  // namespace aq

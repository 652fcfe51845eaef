// Integer product with one weight scale per 128-k group (Sec. 4.4), on the tensor cores.
//
// Every 128-k block is one accumulation of its own (tcgen05.mma kind::i8 into one of two
// accumulator stages in tensor memory) that the epilogue drains, converts, multiplies by the
// group's scale and adds to fp32 partial outputs in registers: two CUDA-core instructions per
// element and group, which is what sets this kernel's pace, not the tensor pipe. The kernel is
// therefore built around the epilogue:
//   * eight epilogue warps (two per tensor-memory lane quarter, half of the token columns each)
//     keep the partial outputs of their 32 channels x BM/2 tokens in registers and run a
//     software pipeline over 32-column chunks: the tensor-memory load of the next chunk (of the
//     same accumulation, or of the next one, whose barrier is looked at without blocking) is in
//     flight while the current chunk is converted and added, so the latency of barrier look,
//     scale read and tensor-memory load is not paid between the arithmetic of two chunks;
//   * work is split evenly: the (tile, k block) pairs of the whole product form one sequence
//     that is cut into as many equal ranges as there are CTAs. A tile whose k range is cut
//     leaves fp32 partial outputs of each piece in scratch; the CTA whose piece arrives last
//     adds all pieces in k order (so the result does not depend on who was last) and writes
//     the outputs. Where that exchange would cost more than the idle tail it removes, or
//     without scratch, ranges are cut at tile boundaries instead.
// Operand roles, weight unpacking into tensor memory, the TMA ring and the bounded waits are
// those of the per-channel kernel (aq_gemm_tensor.cu).
#include <cuda.h>

#include "aq_common.cuh"
#include "aq_tc.cuh"

namespace aq {

namespace {

constexpr int kGWarps = 16;
constexpr int kGThreads = kGWarps * 32;
constexpr int kGFirstUnpack = 4;          // warps 0-3: two TMA producers, two MMA issuers
constexpr int kGFirstEpi = 8;             // warps 4-7: weight unpack; warps 8-15: epilogue
constexpr int kGEpiWarps = 8;
// registers per thread after the roles split; the launch allocates 128 for each of the 512 threads
constexpr int kGRegsControl = 40, kGRegsUnpack = 48, kGRegsEpi = 208;
static_assert(128 * kGRegsControl + 128 * kGRegsUnpack + 256 * kGRegsEpi <= kGThreads * 128,
              "register plan exceeds the launch allocation");
constexpr int kGStages = 5;               // shared-memory ring: activation tile + packed weight block per stage
constexpr int kGScaleSlots = 8;           // ring of the blocks' scales, three deeper than the stage ring
constexpr int kGAcc = 2;                  // accumulator stages
constexpr int kGMaxCtas = 57 * 4;         // one arrival counter byte per CTA in the control block

template <int BM>
struct GSmem {
    static constexpr int kCols = BM / 2;                       // token columns of one epilogue warp
    alignas(1024) uint8_t x[kGStages][BM * 128];               // activation tiles, 128-byte swizzled rows
    alignas(128) uint8_t w[kGStages][kBlockBytes];             // packed weight blocks
    // A block's 128 scales. Slot i % 8 is rewritten for block i + 8, whose copy is issued once the MMAs of
    // block i + 3 are complete, which needs the epilogue to have released block i + 1: its read of slot
    // i % 8 (made before it loads block i's sums) is long done.
    alignas(16) __half sc[kGScaleSlots][kTileN];
    alignas(128) __half ystage[kGEpiWarps][kCols][32];         // fp16 outputs of a warp, token-major, for a TMA store
    alignas(8) uint64_t tma_full[kGStages];
    uint64_t smem_empty[kGStages];
    uint64_t a_full[8], a_empty[8];
    uint64_t acc_full[kGAcc], acc_empty[kGAcc];
    uint64_t epi_meet;                                         // the epilogue warps meet here around a shared tile's count
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
    volatile uint32_t is_last;                                 // shared tile: this CTA's piece arrived last
};

struct GParams {
    int M, K, N, Npad, KB;
    int n_tiles_m, n_tiles;
    int aligned;                   // ranges are cut at tile boundaries: no tile is shared
    const uint8_t* w_packed;
    const __half* w_scales;
    const int32_t* scale_exp;
    __half* y;
    int32_t* acc_dump;
    Control* ctl;
    const float* chan_offset;
    float* scratch;                // [CTA][2][epilogue warp][column][lane] fp32 partial outputs
    int8_t* q_next;
    float next_inv, next_lo, next_hi;
    int next_packed;
    int y_tma;
};

// First (tile, k block) pair, as an index into the whole sequence, of CTA `cta` out of `ctas`.
__device__ __forceinline__ long long g_range_begin(const GParams& p, int cta, int ctas) {
    if (p.aligned) return (long long)p.KB * (((long long)cta * p.n_tiles) / ctas);
    return ((long long)cta * p.n_tiles * p.KB) / ctas;
}
// The CTA whose range holds pair u (ranges not cut at tile boundaries).
__device__ __forceinline__ int g_owner(const GParams& p, long long u, int ctas) {
    return (int)((((u + 1) * ctas) - 1) / ((long long)p.n_tiles * p.KB));
}

__device__ __forceinline__ bool g_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// Waits for the tensor-memory loads in flight. The registers of the chunk that is about to be used are
// passed through, so that no use of them can be scheduled above the wait.
__device__ __forceinline__ void g_wait_ld(uint32_t (&v)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                   "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                   "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :: "memory");
}

__device__ __forceinline__ int g_chain_code(__half hv, float inv, float lo, float hi) {
    const float t = __half2float(hv) * inv;                 // exact: inv is a power of two
    if (t != t) return 0;
    return (int)fminf(fmaxf(rintf(t), lo), hi);
}
// Chaining: a warp's 32 codes of one token (lane = channel) go to the staging row, one byte each or, for
// packed 4-bit codes, two per byte (rows of 16 bytes). All 32 lanes call this together.
__device__ __forceinline__ void g_stage_code(__half* stage, int c, int lane, int code, int packed) {
    if (packed) {
        const int hi = __shfl_down_sync(0xFFFFFFFFu, code, 1);
        if (!(lane & 1)) reinterpret_cast<uint8_t*>(stage)[c * 16 + (lane >> 1)] = (uint8_t)((code & 0xF) | (hi << 4));
    } else {
        reinterpret_cast<int8_t*>(stage)[c * 32 + lane] = (int8_t)code;
    }
}

// OFFSET: add the per-channel term of the zero-point variant. CHAIN: write the next layer's codes instead
// of fp16 outputs. DUMP: also write the int32 sums of every group (test aid).
template <int BM, bool OFFSET, bool CHAIN, bool DUMP>
__global__ void __launch_bounds__(kGThreads, 1)
gemm_grouped_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap y_map,
                    const GParams p) {
    extern __shared__ uint8_t smem_raw[];
    using Smem = GSmem<BM>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    static_assert(BM == 64 || BM == 128 || BM == 192, "token tile");
    constexpr int kCols = Smem::kCols;                   // 32, 64 or 96 columns per epilogue warp
    constexpr int kChunks = kCols / 32;
    constexpr int kAccCols = kGAcc * BM;
    constexpr int kNumASlices = (512 - kAccCols) / kAColsPerStage >= 8 ? 8 : (512 - kAccCols) / kAColsPerStage;
    static_assert(kNumASlices >= 4, "weight-slice ring");
    constexpr int kTmemUsed = kAccCols + kNumASlices * kAColsPerStage;
    constexpr int kTmemCols = kTmemUsed <= 128 ? 128 : kTmemUsed <= 256 ? 256 : 512;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = p.KB;
    const int ctas = (int)gridDim.x, cta = (int)blockIdx.x;
    const long long u_begin = g_range_begin(p, cta, ctas), u_end = g_range_begin(p, cta + 1, ctas);
    const uint32_t n_units = (uint32_t)(u_end - u_begin);
    const int tile_first = (int)(u_begin / KB), kb_first = (int)(u_begin % KB);   // where this CTA's range starts

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGStages; ++s) {
            mbar_init(&sm.tma_full[s], 2);
            mbar_init(&sm.smem_empty[s], 1);
        }
        for (int i = 0; i < kNumASlices; ++i) {
            mbar_init(&sm.a_full[i], 4);
            mbar_init(&sm.a_empty[i], 1);
        }
        for (int a = 0; a < kGAcc; ++a) {
            mbar_init(&sm.acc_full[a], 1);
            mbar_init(&sm.acc_empty[a], kGEpiWarps);
        }
        mbar_init(&sm.epi_meet, kGEpiWarps);
        sm.abort_flag = 0;
        sm.is_last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sm.tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tmem_acc = tmem;
    const uint32_t tmem_a = tmem + kAccCols;
    volatile uint32_t* abort_flag = &sm.abort_flag;

    if (warp < kGFirstUnpack) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kGRegsControl));
        if (warp == 0 || warp == 2) {
            // ------------- TMA producers: warp 0 activation tiles, warp 2 weight blocks and scales
            if (lane == 0) {
                // behind the call's own quantize kernel (programmatic stream serialization) the codes are
                // touched only after that grid has completed; the weight producer does not wait
                if (warp == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
                int tile = tile_first, kb = kb_first;
                int mt = tile % p.n_tiles_m, nt = tile / p.n_tiles_m;
                for (uint32_t it = 0; it < n_units; ++it, ++kb) {
                    if (kb == KB) {
                        kb = 0; ++tile;
                        mt = tile % p.n_tiles_m; nt = tile / p.n_tiles_m;
                    }
                    const int s = (int)(it % kGStages);
                    if (!mbar_wait(&sm.smem_empty[s], ((it / kGStages) & 1u) ^ 1u, abort_flag, 1u)) goto role_done;
                    if (warp == 0) {
                        mbar_arrive_expect_tx(&sm.tma_full[s], BM * 128);
                        tma_load_2d(sm.x[s], &x_map, kb * kTileK, mt * BM, &sm.tma_full[s]);
                    } else {
                        mbar_arrive_expect_tx(&sm.tma_full[s], kBlockBytes + kTileN * 2);
                        tma_load_1d(sm.w[s], p.w_packed + ((size_t)nt * KB + kb) * kBlockBytes, kBlockBytes, &sm.tma_full[s]);
                        tma_load_1d(sm.sc[it % kGScaleSlots], p.w_scales + (size_t)kb * p.Npad + nt * kTileN, kTileN * 2,
                                    &sm.tma_full[s]);
                    }
                }
            }
        } else {
            // ------------- MMA issuers: warp 1 the even, warp 3 the odd k blocks; each block is one accumulation
            if (lane == 0) {
                constexpr uint32_t idesc = idesc_i8(128, BM);
                for (uint32_t it = (uint32_t)(warp >> 1); it < n_units; it += 2) {
                    const int a = (int)(it % kGAcc);
                    const int s = (int)(it % kGStages);
                    const int ai = (int)(it % kNumASlices);
                    if (!mbar_wait(&sm.acc_empty[a], ((it / kGAcc) & 1u) ^ 1u, abort_flag, 2u)) goto role_done;
                    if (!mbar_wait(&sm.a_full[ai], (it / kNumASlices) & 1u, abort_flag, 3u)) goto role_done;
                    tc_fence_after();
                    const uint32_t d_addr = tmem_acc + (uint32_t)(a * BM);
                    const uint32_t a_addr = tmem_a + (uint32_t)(ai * kAColsPerStage);
                    const uint64_t bdesc = smem_desc_sw128(smem_u32(sm.x[s]));
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        tc_mma_i8_ts(d_addr, a_addr + 8 * j, bdesc + (uint64_t)(2 * j), idesc, j > 0 ? 1u : 0u);
                    tc_commit(&sm.a_empty[ai]);
                    tc_commit(&sm.smem_empty[s]);
                    tc_commit(&sm.acc_full[a]);
                }
            }
        }
    } else if (warp < kGFirstEpi) {
        // --------------------------------------------------- weight unpack -> tensor memory
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kGRegsUnpack));
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        int pending = -1;                             // slice whose store has been issued but not published
        for (uint32_t it = 0; it < n_units; ++it) {
            const int s = (int)(it % kGStages);
            const int ai = (int)(it % kNumASlices);
            if (!mbar_wait_warp(&sm.tma_full[s], (it / kGStages) & 1u, abort_flag, 6u)) goto role_done;
            const uint4* src = reinterpret_cast<const uint4*>(sm.w[s]) + r;
            uint4 d[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) d[j] = src[j * kTileN];
            if (pending >= 0) {                       // the previous stores had the loads above to finish
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.a_full[pending]);
            }
            if (!mbar_wait_warp(&sm.a_empty[ai], ((it / kNumASlices) & 1u) ^ 1u, abort_flag, 7u)) goto role_done;
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
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kGRegsEpi));
        const int ew = warp - kGFirstEpi;
        const int quarter = warp & 3;
        const int half = ew >> 2;
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int col0 = half * kCols;
        asm volatile("griddepcontrol.wait;" ::: "memory");               // see the activation producer
        const float pe = __int_as_float((127 + *p.scale_exp) << 23) * 0.0625f;   // 2^e; the sums carry a factor 16
        __half* stage = &sm.ystage[ew][0][0];
        uint32_t it = 0;                              // accumulations of this CTA so far
        uint32_t meet_phase = 0;                      // parity of the next meeting of the epilogue warps
        uint32_t left = n_units;                      // accumulations still to come
        // a segment ends at its tile's last k block (the next one then starts a tile) or with the range
        for (int tile = tile_first, kb0 = kb_first; left > 0; ++tile, kb0 = 0) {
            // ---- one segment: k blocks [kb0, kb1) of one tile
            const int kb1 = (uint32_t)(KB - kb0) < left ? KB : kb0 + (int)left;
            const int n_acc = kb1 - kb0;
            left -= (uint32_t)n_acc;
            const int mt = tile % p.n_tiles_m, nt = tile / p.n_tiles_m;
            const int n = nt * kTileN + r;
            const int m_base = mt * BM + col0;
            const bool n_ok = n < p.N;

            float fsum[kCols];
#pragma unroll
            for (int c = 0; c < kCols; ++c) fsum[c] = 0.0f;
            uint32_t vb[2][32];                       // two chunks of sums: one in use, one in flight

            // the first accumulation of the segment: blocking look, scale, first chunk on its way
            if (!mbar_wait_warp(&sm.acc_full[it & 1u], (it >> 1) & 1u, abort_flag, 9u)) goto role_done;
            tc_fence_after();
            float sg = __half2float(sm.sc[it % kGScaleSlots][r]);
            tc_ld32(tmem_acc + lane_addr + (uint32_t)((it & 1u) * BM + col0), vb[0]);

            for (int g = 0; g < n_acc; g += 2) {
#pragma unroll
                for (int gg = 0; gg < 2; ++gg) {
                    if (g + gg < n_acc) {
                        const uint32_t a_cur = it & 1u;
                        const uint32_t taddr = tmem_acc + lane_addr + (uint32_t)(a_cur * BM + col0);
                        const bool has_next = g + gg + 1 < n_acc;
                        const uint32_t itn = it + 1;
                        float sg_next = 0.0f;
#pragma unroll
                        for (int c = 0; c < kChunks; ++c) {
                            const int q = gg * kChunks + c;          // chunk counter inside the pair: buffer q & 1
                            uint32_t (&cur)[32] = vb[q & 1];
                            uint32_t (&nxt)[32] = vb[(q + 1) & 1];
                            g_wait_ld(cur);
                            bool prefetched = false;
                            if (c == kChunks - 1) {
                                // all of this accumulation's sums are in registers: the stage returns to the MMA
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&sm.acc_empty[a_cur]);
                                if (has_next) {
                                    // a look at the next accumulation without blocking (it is normally complete: the
                                    // MMAs take half of what the epilogue takes); its first chunk is then loaded
                                    // while this chunk is converted
                                    const bool ready = g_test_wait(&sm.acc_full[itn & 1u], (itn >> 1) & 1u);
                                    if (__all_sync(0xFFFFFFFFu, ready ? 1 : 0)) {
                                        tc_fence_after();
                                        sg_next = __half2float(sm.sc[itn % kGScaleSlots][r]);
                                        tc_ld32(tmem_acc + lane_addr + (uint32_t)((itn & 1u) * BM + col0), nxt);
                                        prefetched = true;
                                    }
                                }
                            } else {
                                tc_ld32(taddr + (uint32_t)((c + 1) * 32), nxt);
                            }
                            // one conversion and one FMA per element
#pragma unroll
                            for (int i = 0; i < 32; ++i) fsum[c * 32 + i] = fmaf((float)(int)cur[i], sg, fsum[c * 32 + i]);
                            if constexpr (DUMP) {
                                const int kb = kb0 + g + gg;
#pragma unroll
                                for (int i = 0; i < 32; ++i) {
                                    const int m = m_base + c * 32 + i;
                                    if (n_ok && m < p.M) p.acc_dump[((size_t)m * p.N + n) * KB + kb] = (int)cur[i] >> 4;
                                }
                            }
                            if (c == kChunks - 1 && has_next && !prefetched) {
                                if (!mbar_wait_warp(&sm.acc_full[itn & 1u], (itn >> 1) & 1u, abort_flag, 9u)) goto role_done;
                                tc_fence_after();
                                sg_next = __half2float(sm.sc[itn % kGScaleSlots][r]);
                                tc_ld32(tmem_acc + lane_addr + (uint32_t)((itn & 1u) * BM + col0), nxt);
                            }
                        }
                        sg = sg_next;
                        ++it;
                    }
                }
            }

            // ---- end of the segment
            if (n_acc < KB) {
                // A piece of a shared tile: leave the partial outputs in scratch, count the arrival; the CTA
                // whose piece arrives last adds all pieces in k order and writes the outputs.
                const long long t0 = (long long)tile * KB;
                const int c_first = g_owner(p, t0, ctas), c_last = g_owner(p, t0 + KB - 1, ctas);
                const int which = (t0 + kb0 == u_begin) ? 0 : 1;      // the piece starts where this CTA's range starts
                float* mine = p.scratch + ((size_t)(cta * 2 + which) * kGEpiWarps + ew) * (kCols * 32);
#pragma unroll
                for (int c = 0; c < kCols; ++c) __stcg(mine + c * 32 + lane, fsum[c]);
                __threadfence();
                // (the meetings are mbarrier phases with bounded waits, like every other wait here)
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.epi_meet);
                if (!mbar_wait_warp(&sm.epi_meet, meet_phase, abort_flag, 13u)) goto role_done;
                meet_phase ^= 1u;
                if (ew == 0 && lane == 0) {
                    const unsigned int shift = 8u * (unsigned int)(c_first & 3);
                    const unsigned int old = atomicAdd(&p.ctl->split_flags[c_first >> 2], 1u << shift);
                    sm.is_last = (((old >> shift) & 0xFFu) == (unsigned int)(c_last - c_first)) ? 1u : 0u;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.epi_meet);
                if (!mbar_wait_warp(&sm.epi_meet, meet_phase, abort_flag, 13u)) goto role_done;
                meet_phase ^= 1u;
                if (!sm.is_last) continue;
                __threadfence();
                for (int pc = c_first; pc <= c_last; ++pc) {
                    const long long pb = g_range_begin(p, pc, ctas);
                    const int pwhich = (pb >= t0) ? 0 : 1;            // the piece starts where its CTA's range starts
                    const float* src = p.scratch + ((size_t)(pc * 2 + pwhich) * kGEpiWarps + ew) * (kCols * 32);
                    if (pc == c_first) {
#pragma unroll
                        for (int c = 0; c < kCols; ++c) fsum[c] = __ldcg(src + c * 32 + lane);
                    } else {
#pragma unroll
                        for (int c = 0; c < kCols; ++c) fsum[c] += __ldcg(src + c * 32 + lane);
                    }
                }
            }
            if constexpr (OFFSET) {
                const float off_n = n_ok ? p.chan_offset[n] * 16.0f : 0.0f;      // pe carries the 1/16
#pragma unroll
                for (int c = 0; c < kCols; ++c) fsum[c] += off_n;
            }
            if (p.y_tma) {
                // the previous tile's store must have read the staging rows before they change
                if (lane == 0) tma_store_wait_read();
                __syncwarp();
#pragma unroll
                for (int c = 0; c < kCols; ++c) {
                    const __half hv = __float2half_rn(fsum[c] * pe);
                    if constexpr (CHAIN)
                        g_stage_code(stage, c, lane, g_chain_code(hv, p.next_inv, p.next_lo, p.next_hi), p.next_packed);
                    else
                        stage[c * 32 + lane] = hv;
                }
                fence_proxy_async();
                __syncwarp();
                const int n0 = nt * kTileN + quarter * 32;
                if (lane == 0 && n0 < p.N && m_base < p.M)
                    tma_store_2d(&y_map, stage, (CHAIN && p.next_packed) ? n0 >> 1 : n0, m_base);
            } else {
#pragma unroll
                for (int c = 0; c < kCols; ++c) {
                    const int m = m_base + c;
                    if (n_ok && m < p.M) {
                        const __half hv = __float2half_rn(fsum[c] * pe);
                        if constexpr (CHAIN)
                            p.q_next[(size_t)m * p.N + n] = (int8_t)g_chain_code(hv, p.next_inv, p.next_lo, p.next_hi);
                        else
                            p.y[(size_t)m * p.N + n] = hv;
                    }
                }
            }
        }
    }

role_done:
    if (warp >= kGFirstEpi && lane == 0) tma_store_wait_read();   // staging rows live until read
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols)
                     : "memory");
    }
}

typedef CUresult (*GEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int grouped_token_tile(int M) { return M <= 64 ? 64 : M <= 128 ? 128 : 192; }

// How the sequence of (tile, k block) pairs is cut. Even ranges (shared tiles) when the schedule gets shorter
// by more than the exchange of partial outputs costs (about eight k blocks' time per CTA).
struct GPlan {
    int bm, ctas, aligned;
    size_t scratch_bytes;
};
GPlan grouped_plan(int M, int K, int N, int sm_count, size_t scratch_avail) {
    GPlan pl;
    pl.bm = grouped_token_tile(M);
    const int KB = K / kTileK;
    const long n_tiles = (long)((M + pl.bm - 1) / pl.bm) * (round_up(N, kTileN) / kTileN);
    const int max_ctas = sm_count < kGMaxCtas ? sm_count : kGMaxCtas;
    const size_t per_cta = (size_t)2 * kTileN * pl.bm * sizeof(float);
    // cut at tile boundaries
    const int ctas_aligned = (int)(n_tiles < max_ctas ? n_tiles : max_ctas);
    const long cost_aligned = ((n_tiles + ctas_aligned - 1) / ctas_aligned) * KB;
    // even ranges: with fewer tiles than SMs every tile is shared by as many CTAs as leave each at least four k blocks
    int ctas_even = max_ctas;
    if (n_tiles < max_ctas) {
        int s = (int)(max_ctas / n_tiles);
        if (s > KB / 4) s = KB / 4;
        if (s > 8) s = 8;
        if (s < 1) s = 1;
        ctas_even = (int)n_tiles * s;
    }
    const long cost_even = (n_tiles * KB + ctas_even - 1) / ctas_even + 8;
    const size_t need = (size_t)ctas_even * per_cta;
    if (cost_even < cost_aligned && scratch_avail >= need) {
        pl.ctas = ctas_even; pl.aligned = 0; pl.scratch_bytes = need;
    } else {
        pl.ctas = ctas_aligned; pl.aligned = 1; pl.scratch_bytes = 0;
    }
    return pl;
}

template <int BM, bool OFFSET, bool CHAIN, bool DUMP>
cudaError_t launch_grouped_t(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream, const GPlan& pl) {
    using Smem = GSmem<BM>;
    const size_t smem_bytes = sizeof(Smem) + 1024;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(gemm_grouped_kernel<BM, OFFSET, CHAIN, DUMP>, dev.device, smem_bytes);
        e != cudaSuccess)
        return e;
    GEncodeTiledFn enc = reinterpret_cast<GEncodeTiledFn>(dev.encode_tiled);
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
    const cuuint64_t strides[1] = {(cuuint64_t)a.K};
    const cuuint32_t box[2] = {128u, (cuuint32_t)BM};
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
            const cuuint32_t ybox[2] = {a.next_packed ? 16u : 32u, (cuuint32_t)Smem::kCols};
            if (enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, a.q_next, ydims, ystrides, ybox, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
            y_tma = 1;
        }
    } else if (a.N % 8 == 0 && (reinterpret_cast<uintptr_t>(a.y) & 15u) == 0) {
        const cuuint64_t ydims[2] = {(cuuint64_t)a.N, (cuuint64_t)a.M};
        const cuuint64_t ystrides[1] = {(cuuint64_t)a.N * 2};
        const cuuint32_t ybox[2] = {32u, (cuuint32_t)Smem::kCols};
        if (enc(&ymap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, a.y, ydims, ystrides, ybox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        y_tma = 1;
    }

    GParams p;
    p.M = a.M; p.K = a.K; p.N = a.N; p.Npad = round_up(a.N, kTileN); p.KB = a.K / kTileK;
    p.n_tiles_m = (a.M + BM - 1) / BM;
    p.n_tiles = p.n_tiles_m * (p.Npad / kTileN);
    p.aligned = pl.aligned;
    p.w_packed = a.w_packed; p.w_scales = a.w_scales; p.scale_exp = a.scale_exp;
    p.y = a.y; p.acc_dump = a.acc_dump; p.ctl = a.ctl; p.chan_offset = a.chan_offset;
    p.scratch = a.split_scratch;
    p.q_next = a.q_next;
    p.next_inv = ldexpf(1.0f, -a.next_exp);
    p.next_lo = -(float)(1 << (a.next_bits - 1));
    p.next_hi = (float)((1 << (a.next_bits - 1)) - 1);
    p.next_packed = a.next_packed ? 1 : 0;
    p.y_tma = y_tma;

    // Behind the call's own quantize kernel the launch may overlap that kernel's drain (the kernel waits
    // for it before it reads what it wrote).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.ctas);
    cfg.blockDim = dim3(kGThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.after_quantize ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, gemm_grouped_kernel<BM, OFFSET, CHAIN, DUMP>, map, ymap, p);
}

template <int BM>
cudaError_t launch_grouped_bm(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream, const GPlan& pl) {
    if (a.q_next) {
        if (a.chan_offset) return cudaErrorInvalidValue;       // the two variants are not combined
        return a.acc_dump ? launch_grouped_t<BM, false, true, true>(a, dev, stream, pl)
                          : launch_grouped_t<BM, false, true, false>(a, dev, stream, pl);
    }
    if (a.chan_offset)
        return a.acc_dump ? launch_grouped_t<BM, true, false, true>(a, dev, stream, pl)
                          : launch_grouped_t<BM, true, false, false>(a, dev, stream, pl);
    return a.acc_dump ? launch_grouped_t<BM, false, false, true>(a, dev, stream, pl)
                      : launch_grouped_t<BM, false, false, false>(a, dev, stream, pl);
}

}  // namespace

size_t grouped_scratch_bytes(int M, int K, int N, int sm_count) {
    return grouped_plan(M, K, N, sm_count, ~(size_t)0).scratch_bytes;
}

cudaError_t launch_gemm_grouped(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    const size_t avail = (a.split_scratch && (reinterpret_cast<uintptr_t>(a.split_scratch) & 15u) == 0) ? a.split_bytes : 0;
    const GPlan pl = grouped_plan(a.M, a.K, a.N, dev.sm_count, avail);
    switch (pl.bm) {
        case 64: return launch_grouped_bm<64>(a, dev, stream, pl);
        case 128: return launch_grouped_bm<128>(a, dev, stream, pl);
        default: return launch_grouped_bm<192>(a, dev, stream, pl);
    }
}

}  // namespace aq

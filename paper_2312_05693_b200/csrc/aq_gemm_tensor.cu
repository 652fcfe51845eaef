// Integer product on the 5th-generation tensor cores (tcgen05, kind::i8) with TMEM
// accumulators, for the sums of Sec. 4.4 / Algorithm 1 and the floating-point output.
//
// Operand roles are swapped with respect to y = x w^T: the 128 output channels of a tile
// are the MMA's M dimension and the tokens its N dimension, so that
//   * the 4-bit weights stay packed in shared memory (one contiguous 8 KB bulk copy per
//     128 x 128 block): four warps widen each nibble to the int8 value 16*code with two
//     logic ops per word and store the result straight into tensor memory, where the MMA
//     reads it as its A operand, so the widened weights never take shared-memory bandwidth;
//   * every epilogue thread owns one output channel, so its weight scale(s) sit in a
//     register and the per-128-k group rescaling costs one FMA per element;
//   * the int8 activation tile (tokens x 128 k) is the only shared-memory operand, staged
//     by TMA with the 128-byte swizzle and read through an MMA shared-memory descriptor.
//
// One persistent CTA per SM walks a static list of (channel tile, token tile) pairs.
// Warp roles: 0 and 2 = TMA producers (activations / weights), 1 and 3 = MMA issuers (warp 1
// also owns the TMEM allocation; warp 3 only works in per-group mode), 4-11 = weight unpack
// (two groups of four taking alternate k blocks; only the first group works in per-group mode),
// 12-19 = epilogue; registers are moved from
// the first two roles to the epilogue with setmaxnreg. One thread spends about 55 cycles per
// MMA instruction and about 100 per TMA instruction, which is why issue is spread over
// threads and why the tile is 256 tokens wide where tensor memory allows it. Two (one scale per channel)
// or three (per-group scales) accumulator stages in TMEM let the epilogue of one
// accumulation overlap the MMAs of the next ones. Every wait is bounded; on expiry the CTA records a status
// word, stops issuing work and leaves through the common exit that frees TMEM.
#include <cuda.h>

#include "aq_common.cuh"
#include "aq_tc.cuh"

namespace aq {

namespace {

constexpr int kUnpackGroups = 2;              // groups of four unpack warps; group g takes k blocks g, g+2, ...
constexpr int kFirstUnpackWarp = 4;           // warps 0-3 (one warpgroup): two TMA producers, two MMA issuers
constexpr int kWarps = 20;
constexpr int kThreads = kWarps * 32;
// Registers per thread after the roles split (setmaxnreg works on aligned groups of four warps):
constexpr int kRegsControl = 40, kRegsUnpack = 48;
// The warps behind the control warpgroup are unpack warps, then epilogue warps. Eight epilogue warps (two per
// TMEM lane quarter, half of the token columns each) follow two groups of unpack warps; the per-group
// kernels with 96- or 192-token tiles run twelve (three per quarter, a third of the columns each) behind
// the one unpack group they need: there the per-group rescaling sets the pace, and a third warp per
// scheduler hides the latency of the other two's barrier and tensor-memory round trips.
template <int BM, bool GROUPED>
struct Roles {
    static constexpr int kEpiWarps = (GROUPED && (BM == 96 || BM == 192)) ? 12 : 8;
    static constexpr int kFirstEpiWarp = kWarps - kEpiWarps;
    static constexpr int kRegsEpilogue = kEpiWarps == 12 ? 128 : 168;
    static constexpr int kColsPerEpiWarp = BM / (kEpiWarps / 4);
    // setmaxnreg can only hand out what the launch allocated (96 registers for each of the threads): a
    // larger request would wait forever.
    static_assert(128 * kRegsControl + 32 * (kFirstEpiWarp - kFirstUnpackWarp) * kRegsUnpack +
                          32 * kEpiWarps * kRegsEpilogue <= kThreads * 96,
                  "register plan exceeds the launch allocation");
};
template <int BM>
struct TileConfig {
    // shared-memory ring depth: activation tile + packed weight block (+ scales) per stage
    static constexpr int kNumStages = BM >= 192 ? 5 : 6;
};

template <int BM, int EPI_WARPS>
struct SharedStorage {
    static constexpr int kNumStages = TileConfig<BM>::kNumStages;
    alignas(1024) uint8_t x[kNumStages][BM * 128];   // activation tiles, 128-byte swizzled rows
    alignas(128) uint8_t w[kNumStages][kBlockBytes]; // packed weight blocks (128 channels x 128 k)
    // Weight scales of each block's group (grouped mode), in a ring three slots deeper than the
    // stage ring. A slot is rewritten for block i only after the MMAs of block i - kNumStages
    // completed, which (three accumulator stages) needs the epilogue of every block up to
    // i - kNumStages - 3 to have finished: all reads of the slot's previous content are done.
    static constexpr int kNumScaleSlots = kNumStages + 3;
    alignas(16) __half sc[kNumScaleSlots][kTileN];
    // Each epilogue warp stages fp16 outputs of its 32 channels here, kStageRows tokens at a time
    // (token-major rows of 64 bytes), and hands them to a TMA store.
    static constexpr int kStageRows = BM / (EPI_WARPS / 4) <= 64 ? BM / (EPI_WARPS / 4) : 32;
    alignas(128) __half ystage[EPI_WARPS][kStageRows][32];
    alignas(8) uint64_t tma_full[kNumStages];        // both producers' bytes landed -> unpack warps
    uint64_t smem_empty[kNumStages];                 // MMA done (+ epilogue took the scales) -> TMA producers
    uint64_t a_full[8];                              // unpack warps stored the slice -> MMA
    uint64_t a_empty[8];                             // MMA done with the slice -> unpack warps
    uint64_t acc_full[3];                            // MMA -> epilogue
    uint64_t acc_empty[3];                           // epilogue -> MMA
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
};

struct TensorParams {
    int M, K, N, Npad;
    int n_tiles_m, n_tiles;        // token tiles; total tiles
    const uint8_t* w_packed;
    const __half* w_scales;
    const int32_t* scale_exp;
    __half* y;
    int32_t* acc_dump;
    Control* ctl;
    const float* chan_offset;      // NULL or [N]: per-channel term added before the 2^e factor
    int split_base;                // SPLIT kernels: CTAs 2j and 2j+1 share tile split_base + j, half of K each
    float* split_scratch;          // [shared tile][half][epilogue warp][column][lane] fp32 partial outputs
    int8_t* q_next;                // chaining: the next layer's codes [M][N] are written instead of y
    float next_inv, next_lo, next_hi;   // 2^-next_exp and the code range of the next layer
    int next_packed;               // chaining: 4-bit codes leave two per byte (even channel in the low nibble)
    int y_tma;                     // outputs leave through y_map (needs N % 8 == 0 and a 16-byte aligned y)
};

// The code the next layer's quantizer gives the fp16 output value (static exponent; NaN -> 0).
__device__ __forceinline__ int chain_code(__half hv, float inv, float lo, float hi) {
    const float t = __half2float(hv) * inv;                 // exact: inv is a power of two
    if (t != t) return 0;
    return (int)fminf(fmaxf(rintf(t), lo), hi);
}

// Chaining: a warp's 32 codes of one token (lane = channel) go to the staging row: one byte each, or, for
// packed 4-bit codes, the even lane stores its code and its neighbour's in one byte (rows of 16 bytes).
// All 32 lanes call this together.
__device__ __forceinline__ void stage_code(__half* stage, int c, int lane, int code, int packed) {
    if (packed) {
        const int hi = __shfl_down_sync(0xFFFFFFFFu, code, 1);
        if (!(lane & 1)) reinterpret_cast<uint8_t*>(stage)[c * 16 + (lane >> 1)] = (uint8_t)((code & 0xF) | (hi << 4));
    } else {
        reinterpret_cast<int8_t*>(stage)[c * 32 + lane] = (int8_t)code;
    }
}

// OFFSET: add the per-channel term of the zero-point variant. CHAIN: write the next layer's codes
// instead of fp16 outputs. Separate instantiations, so that the code of the plain kernels does not
// change with them. SPLIT (per-group scales only): the launch covers the tiles of a last, partial round;
// every tile is shared by two CTAs that take half of the k range each, leave fp32 partial sums in
// scratch, and whichever epilogue warp arrives second adds the other's sums and writes the outputs
// (nobody waits).
template <int BM, bool GROUPED, bool OFFSET, bool CHAIN, bool SPLIT = false>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tensor_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap y_map,
                   const TensorParams p) {
    extern __shared__ uint8_t smem_raw[];
    using R = Roles<BM, GROUPED>;
    constexpr int kEpiWarps = R::kEpiWarps, kFirstEpiWarp = R::kFirstEpiWarp, kRegsEpilogue = R::kRegsEpilogue;
    using Smem = SharedStorage<BM, kEpiWarps>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    constexpr int kNumStages = TileConfig<BM>::kNumStages;
    // accumulator stages in tensor memory: three for per-group rescaling, otherwise as many
    // 2 (or 1 for the 256-token tile) as leave room for the weight-slice ring
    constexpr int kNumAcc = GROUPED ? (BM > 128 ? 2 : 3) : (BM >= 256 ? 1 : 2);
    constexpr int kAccStride = BM == 96 ? 128 : BM;   // columns between accumulator stages
    constexpr int kNumMmaThreads = GROUPED ? 2 : 1;   // issuers alternate k blocks when every block has its own accumulator
    constexpr int kAccCols = kNumAcc * kAccStride;
    // the rest of tensor memory (up to 8 slices) is the ring of unpacked weight slices (A operand)
    constexpr int kNumASlices = (512 - kAccCols) / kAColsPerStage >= 8 ? 8 : (512 - kAccCols) / kAColsPerStage;
    static_assert(kNumASlices >= 4 && kNumASlices % kUnpackGroups == 0, "weight-slice ring");
    static_assert(!GROUPED || kNumAcc <= 3, "the scale ring's depth assumes at most three accumulator stages");
    constexpr int kTmemColsUsed = kAccCols + kNumASlices * kAColsPerStage;
    constexpr int kTmemCols = kTmemColsUsed <= 128 ? 128 : kTmemColsUsed <= 256 ? 256 : 512;
    static_assert(kTmemColsUsed <= 512, "tensor memory has 512 columns");
    static_assert(BM % 32 == 0 && BM >= 64 && BM <= 256, "token tile");
    constexpr int kColsPerEpiWarp = R::kColsPerEpiWarp;   // each quarter's columns are split between two or three warps
    static_assert(kColsPerEpiWarp % 16 == 0 && (!GROUPED || kColsPerEpiWarp % 32 == 0), "epilogue chunking");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int KB = k_blocks(p.K);      // a last block that K does not fill: zero weight codes meet the tensor map's zero fill
    static_assert(!SPLIT || (GROUPED && !OFFSET && !CHAIN), "only the plain per-group kernel shares tiles");
    const int my_tiles = SPLIT ? 1
                               : (p.n_tiles > (int)blockIdx.x
                                      ? (p.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0);
    // the k blocks of a work item: all of them, or one half when the tile is shared
    const int kb_first = SPLIT ? (((int)blockIdx.x & 1) ? KB / 2 : 0) : 0;
    const int kb_last = SPLIT ? (((int)blockIdx.x & 1) ? KB : KB / 2) : KB;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kNumStages; ++s) {
            mbar_init(&sm.tma_full[s], 2);
            mbar_init(&sm.smem_empty[s], 1);
        }
        for (int i = 0; i < kNumASlices; ++i) {
            mbar_init(&sm.a_full[i], 4);
            mbar_init(&sm.a_empty[i], 1);
        }
        for (int a = 0; a < kNumAcc; ++a) {
            mbar_init(&sm.acc_full[a], 1);
            mbar_init(&sm.acc_empty[a], kEpiWarps);
        }
        sm.abort_flag = 0;
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
    const uint32_t tmem_acc = tmem;                 // columns [0, kNumAcc*BM)
    const uint32_t tmem_a = tmem + kAccCols;        // then kNumASlices slices of 32 columns
    volatile uint32_t* abort_flag = &sm.abort_flag;

    if (warp < kFirstUnpackWarp) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsControl));
      if (warp == 0 || warp == 2) {
        // ------------- TMA producers: warp 0 streams activation tiles, warp 2 weight blocks (+ scales)
        if (lane == 0) {
            // Launched behind the call's own quantize kernel with programmatic stream serialization, this
            // grid is set up while that one drains: the codes (and, in the epilogue, the exponent and the
            // offsets) are touched only after it has completed; the weight producer does not wait. A no-op
            // for a normal launch.
            if (warp == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
            uint32_t it = 0;
            for (int tl = 0; tl < my_tiles; ++tl) {
                const int tile = SPLIT ? p.split_base + ((int)blockIdx.x >> 1) : (int)(blockIdx.x + tl * gridDim.x);
                const int mt = tile % p.n_tiles_m, nt = tile / p.n_tiles_m;
                const uint8_t* wsrc = p.w_packed + (size_t)nt * KB * kBlockBytes;
                for (int kb = kb_first; kb < kb_last; ++kb, ++it) {
                    const int s = (int)(it % kNumStages);
                    const uint32_t ph = (it / kNumStages) & 1u;
                    if (!mbar_wait(&sm.smem_empty[s], ph ^ 1u, abort_flag, 1u)) goto role_done;
                    if (warp == 0) {
                        mbar_arrive_expect_tx(&sm.tma_full[s], BM * 128);
                        tma_load_2d(sm.x[s], &x_map, kb * kTileK, mt * BM, &sm.tma_full[s]);
                    } else {
                        mbar_arrive_expect_tx(&sm.tma_full[s], kBlockBytes + (GROUPED ? kTileN * 2 : 0));
                        tma_load_1d(sm.w[s], wsrc + (size_t)kb * kBlockBytes, kBlockBytes, &sm.tma_full[s]);
                        if (GROUPED)
                            tma_load_1d(sm.sc[it % Smem::kNumScaleSlots],
                                        p.w_scales + (size_t)kb * p.Npad + nt * kTileN, kTileN * 2, &sm.tma_full[s]);
                    }
                }
            }
        }
      } else {
        // ------------- MMA issuers: warp 1 (and warp 3 in grouped mode, taking the odd k blocks)
        const int mma_id = warp >> 1;                  // 0 or 1
        if (lane == 0 && mma_id < kNumMmaThreads) {
            constexpr uint32_t idesc = idesc_i8(128, BM);
            const uint32_t total_iters = (uint32_t)my_tiles * (uint32_t)(kb_last - kb_first);
            if (GROUPED) {
                // every k block is one accumulation into its own accumulator stage
                for (uint32_t it = mma_id; it < total_iters; it += kNumMmaThreads) {
                    const int a = (int)(it % kNumAcc);
                    const int s = (int)(it % kNumStages);
                    const int ai = (int)(it % kNumASlices);
                    if (!mbar_wait(&sm.acc_empty[a], ((it / kNumAcc) & 1u) ^ 1u, abort_flag, 2u)) goto role_done;
                    if (!mbar_wait(&sm.a_full[ai], (it / kNumASlices) & 1u, abort_flag, 3u)) goto role_done;
                    tc_fence_after();
                    const uint32_t d_addr = tmem_acc + (uint32_t)(a * kAccStride);
                    const uint32_t a_addr = tmem_a + (uint32_t)(ai * kAColsPerStage);
                    const uint64_t bdesc = smem_desc_sw128(smem_u32(sm.x[s]));
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        tc_mma_i8_ts(d_addr, a_addr + 8 * j, bdesc + (uint64_t)(2 * j), idesc, j > 0 ? 1u : 0u);
                    tc_commit(&sm.a_empty[ai]);
                    tc_commit(&sm.smem_empty[s]);
                    tc_commit(&sm.acc_full[a]);
                }
            } else {
                uint32_t it = 0;
                for (int tl = 0; tl < my_tiles; ++tl) {
                    const int a = (int)((uint32_t)tl % kNumAcc);
                    const uint32_t aph = ((uint32_t)tl / kNumAcc) & 1u;
                    if (!mbar_wait(&sm.acc_empty[a], aph ^ 1u, abort_flag, 4u)) goto role_done;
                    for (int kb = 0; kb < KB; ++kb, ++it) {
                        const int s = (int)(it % kNumStages);
                        const int ai = (int)(it % kNumASlices);
                        // the unpack warps publish a slice only after the stage's TMA bytes (activation
                        // tile included) have landed, so this one wait covers both operands
                        if (!mbar_wait(&sm.a_full[ai], (it / kNumASlices) & 1u, abort_flag, 5u)) goto role_done;
                        tc_fence_after();
                        const uint32_t d_addr = tmem_acc + (uint32_t)(a * kAccStride);
                        const uint32_t a_addr = tmem_a + (uint32_t)(ai * kAColsPerStage);
                        const uint64_t bdesc = smem_desc_sw128(smem_u32(sm.x[s]));
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            // 32 k per instruction: 8 TMEM columns of A, 32 bytes along the swizzled row of B
                            tc_mma_i8_ts(d_addr, a_addr + 8 * j, bdesc + (uint64_t)(2 * j), idesc,
                                         (kb == 0 && j == 0) ? 0u : 1u);
                        }
                        tc_commit(&sm.a_empty[ai]);
                        tc_commit(&sm.smem_empty[s]);
                    }
                    tc_commit(&sm.acc_full[a]);
                }
            }
        }
      }
    } else if (warp < kFirstEpiWarp) {
        // --------------------------------------------------- weight unpack -> tensor memory
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsUnpack));
        const int quarter = warp & 3;
        const int group = (warp - kFirstUnpackWarp) >> 2;
        const int r = quarter * 32 + lane;            // row inside the 128-channel tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const uint32_t total_iters = (uint32_t)my_tiles * (uint32_t)(kb_last - kb_first);
        int pending = -1;                             // slice whose store has been issued but not published
        // With per-group rescaling the epilogue sets the pace (about four times the MMA time per k block) and
        // one group of unpack warps keeps up; the second group would only poll barriers on the schedulers
        // the epilogue warps issue from (measured: 1-2 % slower with it), so it leaves at once.
        constexpr int kActiveGroups = GROUPED ? 1 : kUnpackGroups;
        if (group >= kActiveGroups) goto role_done;
        for (uint32_t it = group; it < total_iters; it += kActiveGroups) {
            const int s = (int)(it % kNumStages);
            const int ai = (int)(it % kNumASlices);
            if (!mbar_wait_warp(&sm.tma_full[s], (it / kNumStages) & 1u, abort_flag, 6u)) goto role_done;
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
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsEpilogue));
        const int quarter = warp & 3;
        const int half = (warp - kFirstEpiWarp) >> 2;                                // which half (third) of the token columns
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int col0 = half * kColsPerEpiWarp;
        asm volatile("griddepcontrol.wait;" ::: "memory");               // see the activation producer
        const float pe = __int_as_float((127 + *p.scale_exp) << 23);     // 2^e
        [[maybe_unused]] const int G = GROUPED ? KB : 1;
        uint32_t unit = 0;
        [[maybe_unused]] uint32_t g_a = 0, g_ph = 0, g_slot = 0;   // per-group mode: accumulator stage, its parity, scale slot
        for (int tl = 0; tl < my_tiles; ++tl) {
            const int tile = SPLIT ? p.split_base + ((int)blockIdx.x >> 1) : (int)(blockIdx.x + tl * gridDim.x);
            const int mt = tile % p.n_tiles_m, nt = tile / p.n_tiles_m;
            const int n = nt * kTileN + r;
            const int m_base = mt * BM + col0;
            const bool n_ok = n < p.N;
            if constexpr (!GROUPED) {
                const int a = (int)(unit % kNumAcc);
                const uint32_t aph = (unit / kNumAcc) & 1u;
                const float sc = __half2float(p.w_scales[n]) * 0.0625f * pe;   // sums carry a factor 16
                [[maybe_unused]] float off_pe = 0.0f;
                if constexpr (OFFSET) off_pe = (n_ok ? p.chan_offset[n] : 0.0f) * pe;
                if (!mbar_wait_warp(&sm.acc_full[a], aph, abort_flag, 8u)) goto role_done;
                tc_fence_after();
                // all of this warp's sums go to registers and the accumulator returns to the MMA at once,
                // so that the conversion and the stores below overlap the next tile's MMAs
                uint32_t v[kColsPerEpiWarp];
#pragma unroll
                for (int c0 = 0; c0 < kColsPerEpiWarp; c0 += 32)
                    tc_ld32(tmem_acc + lane_addr + (uint32_t)(a * kAccStride + col0 + c0), *reinterpret_cast<uint32_t(*)[32]>(&v[c0]));
                tc_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.acc_empty[a]);
                if (p.y_tma) {
                    __half* stage = &sm.ystage[warp - kFirstEpiWarp][0][0];
                    const int n0 = nt * kTileN + quarter * 32;
#pragma unroll
                    for (int r0 = 0; r0 < kColsPerEpiWarp; r0 += Smem::kStageRows) {
                        if (lane == 0) tma_store_wait_read();     // the previous store has read the staging rows
                        __syncwarp();
#pragma unroll
                        for (int c = 0; c < Smem::kStageRows; ++c) {
                            const __half hv = __float2half_rn(OFFSET ? fmaf((float)(int)v[r0 + c], sc, off_pe)
                                                                     : (float)(int)v[r0 + c] * sc);
                            if constexpr (CHAIN)
                                stage_code(stage, c, lane, chain_code(hv, p.next_inv, p.next_lo, p.next_hi), p.next_packed);
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
                    for (int c = 0; c < kColsPerEpiWarp; ++c) {
                        const int m = m_base + c;
                        if (n_ok && m < p.M) {
                            const __half hv =
                                __float2half_rn(OFFSET ? fmaf((float)(int)v[c], sc, off_pe) : (float)(int)v[c] * sc);
                            if constexpr (CHAIN)
                                p.q_next[(size_t)m * p.N + n] = (int8_t)chain_code(hv, p.next_inv, p.next_lo, p.next_hi);
                            else
                                p.y[(size_t)m * p.N + n] = hv;
                        }
                    }
                }
                if (p.acc_dump) {
#pragma unroll
                    for (int c = 0; c < kColsPerEpiWarp; ++c) {
                        const int m = m_base + c;
                        if (n_ok && m < p.M) p.acc_dump[(size_t)m * p.N + n] = (int)v[c] >> 4;
                    }
                }
                ++unit;
            } else {
                float fsum[kColsPerEpiWarp];                             // fp32 partial outputs
#pragma unroll
                for (int c = 0; c < kColsPerEpiWarp; ++c) fsum[c] = 0.0f;
                for (int kb = kb_first; kb < kb_last; ++kb) {
                    // ring positions are carried in counters (g_a, g_ph, g_slot): no division per block
                    const int a = (int)g_a;
                    if (!mbar_wait_warp(&sm.acc_full[a], g_ph, abort_flag, 9u)) goto role_done;
                    tc_fence_after();
                    // This block's MMAs are complete, so its stage (scales included) had landed: the
                    // issuer saw the unpack warps' signal, which they gave after seeing the TMA barrier.
                    const float sg = __half2float(sm.sc[g_slot][r]) * 0.0625f;
                    if (++g_a == (uint32_t)kNumAcc) { g_a = 0; g_ph ^= 1u; }
                    if (++g_slot == (uint32_t)Smem::kNumScaleSlots) g_slot = 0;
                    static_assert(kColsPerEpiWarp == 32 || kColsPerEpiWarp == 64, "epilogue register plan");
                    const uint32_t taddr = tmem_acc + lane_addr + (uint32_t)(a * kAccStride + col0);
                    // With twelve epilogue warps (128 registers each) a warp's 64 columns pass through one
                    // 32-register buffer in two turns; otherwise all of them are loaded at once.
                    constexpr int kLdCols = (kEpiWarps == 12 && kColsPerEpiWarp == 64) ? 32 : kColsPerEpiWarp;
#pragma unroll
                    for (int c0 = 0; c0 < kColsPerEpiWarp; c0 += kLdCols) {
                        uint32_t v[kLdCols];
                        tc_ld32(taddr + c0, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                        if (kLdCols == 64) tc_ld32(taddr + c0 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32 % kLdCols]));
                        tc_wait_ld();
                        if (c0 + kLdCols == kColsPerEpiWarp) {
                            // the sums are in registers: the accumulator stage goes back to the MMA at once
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&sm.acc_empty[a]);
                        }
#pragma unroll
                        for (int c = 0; c < kLdCols; ++c) {
                            // One conversion and one FMA per element. (An integer add of the bits of
                            // 1.5 * 2^23 plus a float subtract also converts, on the FMA and ALU pipes, but
                            // costs a third instruction; measured 8-16 % slower: issue slots are what this
                            // loop runs out of, not the conversion unit.)
                            fsum[c0 + c] = fmaf((float)(int)v[c], sg, fsum[c0 + c]);
                        }
                        if (p.acc_dump) {
#pragma unroll
                            for (int c = 0; c < kLdCols; ++c) {
                                const int m = m_base + c0 + c;
                                if (n_ok && m < p.M) p.acc_dump[((size_t)m * p.N + n) * G + kb] = (int)v[c] >> 4;
                            }
                        }
                    }
                }
                [[maybe_unused]] bool emit = true;
                if constexpr (SPLIT) {
                    const int ew = warp - kFirstEpiWarp, slot = (int)blockIdx.x >> 1, hf = (int)blockIdx.x & 1;
                    float* mine = p.split_scratch + ((size_t)(slot * 2 + hf) * kEpiWarps + ew) * (kColsPerEpiWarp * 32);
                    const float* other = p.split_scratch + ((size_t)(slot * 2 + (hf ^ 1)) * kEpiWarps + ew) * (kColsPerEpiWarp * 32);
#pragma unroll
                    for (int c = 0; c < kColsPerEpiWarp; ++c) __stcg(mine + c * 32 + lane, fsum[c]);
                    __threadfence();
                    __syncwarp();
                    const int bit_index = slot * kEpiWarps + ew;
                    unsigned int old = 0;
                    if (lane == 0) old = atomicOr(&p.ctl->split_flags[bit_index >> 5], 1u << (bit_index & 31));
                    old = __shfl_sync(0xFFFFFFFFu, old, 0);
                    emit = ((old >> (bit_index & 31)) & 1u) != 0;
                    if (emit) {
                        __threadfence();
#pragma unroll
                        for (int c = 0; c < kColsPerEpiWarp; ++c) fsum[c] += __ldcg(other + c * 32 + lane);
                    }
                }
                if constexpr (OFFSET) {                                  // read after the k loop
                    const float off_n = n_ok ? p.chan_offset[n] : 0.0f;
#pragma unroll
                    for (int c = 0; c < kColsPerEpiWarp; ++c) fsum[c] += off_n;
                }
                if (SPLIT && !emit) {
                    // the other CTA's warp writes this tile's outputs
                } else if (p.y_tma) {
                    static_assert(Smem::kStageRows == kColsPerEpiWarp, "per-group kernels stage a warp's whole tile");
                    // the previous tile's store must have read the staging rows before they change
                    __half* stage = &sm.ystage[warp - kFirstEpiWarp][0][0];
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
#pragma unroll
                    for (int c = 0; c < kColsPerEpiWarp; ++c) {
                        const __half hv = __float2half_rn(fsum[c] * pe);
                        if constexpr (CHAIN)
                            stage_code(stage, c, lane, chain_code(hv, p.next_inv, p.next_lo, p.next_hi), p.next_packed);
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
                    for (int c = 0; c < kColsPerEpiWarp; ++c) {
                        const int m = m_base + c;
                        if (n_ok && m < p.M) {
                            const __half hv = __float2half_rn(fsum[c] * pe);
                            if constexpr (CHAIN)
                                p.q_next[(size_t)m * p.N + n] = (int8_t)chain_code(hv, p.next_inv, p.next_lo, p.next_hi);
                            else
                                p.y[(size_t)m * p.N + n] = hv;
                        }
                    }
                }
            }
        }
    }

role_done:
    if (warp >= kFirstEpiWarp && lane == 0) tma_store_wait_read();   // staging rows live until read
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (sm.abort_flag) {
        // Give copies that may still be in flight time to land before shared memory is released.
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
        if (threadIdx.x == 0) atomicCAS(&p.ctl->status, 0u, sm.abort_flag);   // the first CTA to give up names its wait
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// Rate probe: what this GPU's tensor cores deliver on kind::i8 when nothing else is in the way.
// One CTA per SM; one thread issues `iters` rounds of four 128 x 256 x 32 MMAs on operands that
// stay where they are (pseudo-random bytes, so that the data toggles as real codes do): both from
// shared memory, or A from tensor memory as in the product kernel. No loads, no epilogue. Batches
// of 32 rounds are committed to two alternating barriers and the issuer stays one batch ahead,
// so the pipe never drains and the queue stays bounded.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void tc_mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

struct ProbeSmem {
    alignas(1024) uint8_t a[128 * 128];     // 128 rows x 128 k, 128-byte swizzled rows
    alignas(1024) uint8_t b[256 * 128];     // 256 rows x 128 k
    alignas(8) uint64_t bar[2];
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
};

__global__ void __launch_bounds__(128, 1) int8_probe_kernel(int iters, int a_from_tmem, Control* ctl) {
    extern __shared__ uint8_t smem_raw[];
    ProbeSmem& sm = *reinterpret_cast<ProbeSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t* words = reinterpret_cast<uint32_t*>(sm.a);
    for (int i = threadIdx.x; i < (int)(sizeof(sm.a) + sizeof(sm.b)) / 4; i += blockDim.x) {
        uint32_t v = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;       // any bytes will do
        v ^= v >> 15; v *= 2246822519u; v ^= v >> 13;
        words[i] = v;
    }
    fence_proxy_async();
    if (threadIdx.x == 0) {
        mbar_init(&sm.bar[0], 1);
        mbar_init(&sm.bar[1], 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&sm.tmem_base)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tmem_a = tmem + 256;            // after the 256 accumulator columns
    if (a_from_tmem) {                             // 128 lanes x 32 columns of bytes for the A operand
        uint32_t v[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = words[(threadIdx.x * 32 + j * 8 + i) & 4095];
            tc_st8(tmem_a + ((uint32_t)(warp * 32) << 16) + 8 * j, v);
        }
        tc_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0 && lane == 0) {
        constexpr uint32_t idesc = idesc_i8(128, 256);
        constexpr int kBatch = 32;
        const uint64_t adesc = smem_desc_sw128(smem_u32(sm.a)), bdesc = smem_desc_sw128(smem_u32(sm.b));
        const int batches = (iters + kBatch - 1) / kBatch;
        bool ok = true;
        for (int bt = 0; bt < batches && ok; ++bt) {
            if (bt >= 2) ok = mbar_wait(&sm.bar[bt & 1], (uint32_t)((bt >> 1) - 1) & 1u, &sm.abort_flag, 12u);
            if (!ok) break;
            const int n = min(kBatch, iters - bt * kBatch);
            for (int it = 0; it < n; ++it) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (a_from_tmem) tc_mma_i8_ts(tmem, tmem_a + 8 * j, bdesc + (uint64_t)(2 * j), idesc, 1u);
                    else tc_mma_i8_ss(tmem, adesc + (uint64_t)(2 * j), bdesc + (uint64_t)(2 * j), idesc, 1u);
                }
            }
            tc_commit(&sm.bar[bt & 1]);
        }
        // drain: the last one or two batches
        for (int bt = max(batches - 2, 0); bt < batches && ok; ++bt)
            ok = mbar_wait(&sm.bar[bt & 1], (uint32_t)(bt >> 1) & 1u, &sm.abort_flag, 12u);
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (sm.abort_flag && threadIdx.x == 0) atomicCAS(&ctl->status, 0u, sm.abort_flag);
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

// Shared tiles pay from K = 8192 on with 64- and 128-token tiles and from K = 4096 on with 192-token
// tiles, where half a tile is worth more (see launch_bm).
constexpr int split_min_k_blocks(int bm) { return bm >= 192 ? 32 : 64; }

// Whether a last, partial round of `rem` tiles is run as shared tiles.
inline bool round_is_shared(int rem, int sms, int k_blocks, int bm) {
    return rem > 0 && 2 * rem <= sms && k_blocks >= split_min_k_blocks(bm) && rem <= Control::kMaxSplitTiles;
}

// Token tile of the per-group kernels. Up to 64 tokens: 64. Otherwise 128 (eight epilogue warps, three
// accumulator stages) or 192 (twelve epilogue warps, two stages), whichever gives the shorter schedule:
// rounds of tiles over the SMs (a shared last round counts half) x tile height x the measured cost per
// token column and k block (about 7.6 cycles with 128-token tiles, 6.6 with 192-token tiles).
int grouped_token_tile(int M, int K, int N, int sms, bool may_share) {
    if (M <= 64) return 64;
    const int kbs = K / kTileK, n_tiles_n = round_up(N, kTileN) / kTileN;
    auto cost = [&](int bm, float per_col) {
        const long tiles = (long)((M + bm - 1) / bm) * n_tiles_n;
        const long rounds = tiles / sms;
        const int rem = (int)(tiles % sms);
        const float last = rem == 0 ? 0.0f : (may_share && round_is_shared(rem, sms, kbs, bm) ? 0.5f : 1.0f);
        return ((float)rounds + last) * (float)bm * per_col;
    };
    return cost(192, 6.6f) < cost(128, 7.6f) ? 192 : 128;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// tile_limit >= 0: only the first tile_limit tiles (whole rounds). SPLIT: the tiles from split_base on, two CTAs each.
template <int BM, bool GROUPED, bool OFFSET, bool CHAIN, bool SPLIT = false>
cudaError_t launch_off(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream, int tile_limit = -1,
                       int split_base = 0, int split_tiles = 0) {
    using Smem = SharedStorage<BM, Roles<BM, GROUPED>::kEpiWarps>;
    const size_t smem_bytes = sizeof(Smem) + 1024;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(gemm_tensor_kernel<BM, GROUPED, OFFSET, CHAIN, SPLIT>, dev.device, smem_bytes);
        e != cudaSuccess)
        return e;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
    const cuuint64_t strides[1] = {(cuuint64_t)a.K};
    const cuuint32_t box[2] = {128u, (cuuint32_t)BM};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(dev.encode_tiled)(
        &map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(a.q), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;

    CUtensorMap ymap = map;   // placeholder when the store path is off
    int y_tma = 0;
    if (CHAIN) {
        // the staged rows hold one byte per value (or per two values when packed): a map over the code
        // matrix, 32-byte (16-byte) rows
        if (a.next_packed && (a.N % 32 != 0 || (reinterpret_cast<uintptr_t>(a.q_next) & 15u) != 0))
            return cudaErrorInvalidValue;                    // packed codes only leave through the TMA store
        if (a.N % 16 == 0 && (reinterpret_cast<uintptr_t>(a.q_next) & 15u) == 0) {
            const cuuint64_t row_bytes = a.next_packed ? (cuuint64_t)a.N / 2 : (cuuint64_t)a.N;
            const cuuint64_t ydims[2] = {row_bytes, (cuuint64_t)a.M};
            const cuuint64_t ystrides[1] = {row_bytes};
            const cuuint32_t ybox[2] = {a.next_packed ? 16u : 32u, (cuuint32_t)Smem::kStageRows};
            const CUresult ry = reinterpret_cast<EncodeTiledFn>(dev.encode_tiled)(
                &ymap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, a.q_next, ydims, ystrides, ybox, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (ry != CUDA_SUCCESS) return cudaErrorInvalidValue;
            y_tma = 1;
        }
    } else if (a.N % 8 == 0 && (reinterpret_cast<uintptr_t>(a.y) & 15u) == 0) {
        const cuuint64_t ydims[2] = {(cuuint64_t)a.N, (cuuint64_t)a.M};
        const cuuint64_t ystrides[1] = {(cuuint64_t)a.N * 2};
        const cuuint32_t ybox[2] = {32u, (cuuint32_t)Smem::kStageRows};
        const CUresult ry = reinterpret_cast<EncodeTiledFn>(dev.encode_tiled)(
            &ymap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, a.y, ydims, ystrides, ybox, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (ry != CUDA_SUCCESS) return cudaErrorInvalidValue;
        y_tma = 1;
    }

    TensorParams p;
    p.y_tma = y_tma;
    p.M = a.M; p.K = a.K; p.N = a.N; p.Npad = round_up(a.N, kTileN);
    p.n_tiles_m = (a.M + BM - 1) / BM;
    p.n_tiles = p.n_tiles_m * (p.Npad / kTileN);
    p.w_packed = a.w_packed; p.w_scales = a.w_scales; p.scale_exp = a.scale_exp;
    p.y = a.y; p.acc_dump = a.acc_dump; p.ctl = a.ctl; p.chan_offset = a.chan_offset;
    p.q_next = a.q_next;
    p.next_inv = ldexpf(1.0f, -a.next_exp);
    p.next_lo = -(float)(1 << (a.next_bits - 1));
    p.next_hi = (float)((1 << (a.next_bits - 1)) - 1);
    p.next_packed = a.next_packed ? 1 : 0;
    if (tile_limit >= 0) p.n_tiles = tile_limit;
    p.split_base = split_base;
    p.split_scratch = a.split_scratch;
    const int grid = SPLIT ? 2 * split_tiles : (p.n_tiles < dev.sm_count ? p.n_tiles : dev.sm_count);
    if constexpr (SPLIT) {
        // This launch depends on nothing the preceding whole-round launch writes (other tiles of y; the
        // partial sums and their flags are its own), so it may be set up while that one still runs: its
        // CTAs start as SMs become free instead of after a launch gap.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = split_base > 0 ? 1 : 0;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, gemm_tensor_kernel<BM, GROUPED, OFFSET, CHAIN, SPLIT>, map, ymap, p);
    } else {
        // Behind the call's own quantize kernel the launch may overlap that kernel's drain (the kernel
        // waits for it before it reads what it wrote).
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = a.after_quantize ? 1 : 0;
        return cudaLaunchKernelEx(&cfg, gemm_tensor_kernel<BM, GROUPED, OFFSET, CHAIN, SPLIT>, map, ymap, p);
    }
}

template <int BM, bool GROUPED>
cudaError_t launch_bm(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    if (a.q_next) {
        if (a.chan_offset) return cudaErrorInvalidValue;       // the two variants are not combined
        return launch_off<BM, GROUPED, false, true>(a, dev, stream);
    }
    if (a.chan_offset) return launch_off<BM, GROUPED, true, false>(a, dev, stream);
    if constexpr (GROUPED) {
        // A last round that would leave more than half of the SMs idle is run as shared tiles, when the
        // reduction is deep enough for half a tile to outweigh the second launch and the exchange of
        // partial sums (measured with 128-token tiles: a loss of 2-5 us at K = 4096, a gain of 8 us at
        // K = 11008; with 192-token tiles a gain of 2 us at K = 4096 already).
        const int sms = dev.sm_count;
        const int n_tiles = ((a.M + BM - 1) / BM) * (round_up(a.N, kTileN) / kTileN);
        const int rounds = n_tiles / sms, rem = n_tiles % sms;
        const size_t need = (size_t)rem * 2 * BM * kTileN * sizeof(float);
        if (round_is_shared(rem, sms, a.K / kTileK, BM) && a.split_scratch &&
            a.split_bytes >= need && (reinterpret_cast<uintptr_t>(a.split_scratch) & 15u) == 0) {
            if (rounds > 0) {
                const cudaError_t e = launch_off<BM, true, false, false>(a, dev, stream, rounds * sms);
                if (e != cudaSuccess) return e;
            }
            return launch_off<BM, true, false, false, true>(a, dev, stream, -1, rounds * sms, rem);
        }
    }
    return launch_off<BM, GROUPED, false, false>(a, dev, stream);
}

}  // namespace

size_t tensor_split_scratch_bytes(int M, int K, int N, int group, int sm_count) {
    if (!group) return 0;
    const int bm = grouped_token_tile(M, K, N, sm_count, true);
    const int n_tiles = ((M + bm - 1) / bm) * (round_up(N, kTileN) / kTileN);
    const int rem = n_tiles % sm_count;
    if (!round_is_shared(rem, sm_count, K / kTileK, bm)) return 0;
    return (size_t)rem * 2 * bm * kTileN * sizeof(float);
}

cudaError_t launch_int8_probe(int iters, int a_from_tmem, Control* ctl, const DeviceInfo& dev, cudaStream_t stream) {
    const size_t smem_bytes = sizeof(ProbeSmem) + 1024;
    static SmemOptIn opt_in;
    if (const cudaError_t e = opt_in.ensure(int8_probe_kernel, dev.device, smem_bytes); e != cudaSuccess) return e;
    int8_probe_kernel<<<dev.sm_count, 128, smem_bytes, stream>>>(iters, a_from_tmem, ctl);
    return cudaGetLastError();
}

cudaError_t launch_gemm_tensor(const GemmArgs& a, const DeviceInfo& dev, cudaStream_t stream) {
    if (a.M <= 64) return a.group ? launch_bm<64, true>(a, dev, stream) : launch_bm<64, false>(a, dev, stream);
    if (a.group) {
        // the chained and zero-point variants have no shared-tile launch
        switch (grouped_token_tile(a.M, a.K, a.N, dev.sm_count, !a.q_next && !a.chan_offset)) {
            case 96: return launch_bm<96, true>(a, dev, stream);
            case 192: return launch_bm<192, true>(a, dev, stream);
            default: return launch_bm<128, true>(a, dev, stream);
        }
    }
    // one scale per channel: two channel blocks share a 128-token activation tile where the shape allows it
    if (gemm_wide_applies(a)) return launch_gemm_wide(a, dev, stream);
    // one scale per channel: the 256-token tile halves the MMA instructions per unit of work
    if (a.M <= 128) return launch_bm<128, false>(a, dev, stream);
    return launch_bm<256, false>(a, dev, stream);
}

}  // namespace aq

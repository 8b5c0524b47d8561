// Channel-compacted FFN on the 5th-generation tensor cores (Section 4.6):
//   Y = gelu(X . W1[:, N]) . W2[N, :]   for the present rows of every sample.
//
// One persistent CTA per SM walks tiles of 128 present rows (row table in ffn_plan.cuh).
// Per tile and per chunk of CH kept channels (CH = 256, or 128 when d_model = 384):
//   GEMM1  H[128 x CH] = X_tile[128 x D] . W1c_chunk^T            (tcgen05, fp32 in TMEM)
//   epilogue  H -> gelu -> bf16 -> shared memory (K-major, 128-byte swizzle)
//   GEMM2  Y[128 x D] += H[128 x CH] . W2c_chunk                  (tcgen05, fp32 in TMEM)
// The hidden activations never leave the SM.  Weights are the gathered, K-major copies made
// by the prepare kernel and stream through a ring of 32 KB TMA stages; every stage feeds
// 512 tensor-pipe cycles (four N=256 or eight N=128 instructions), which is what it takes to
// hide the fixed cost of a stage hand-over (an mbarrier wait, the copy issue, a commit) behind
// the arithmetic.  Two producer threads share the ring for the same reason.  X rows are
// gathered with 16-byte async copies, one 64-column block at a time, into the swizzled layout
// TMA would produce; a block's slot is refilled for the next tile as soon as the last chunk's
// GEMM1 has read it.
//
// The tensor pipe is kept busy across chunk and tile boundaries: the issuer runs GEMM1 of the
// next chunk (or of the next tile's first chunk) before GEMM2 of the current one, so GEMM2
// never waits for the GELU epilogue with nothing else queued.
//
// With d_model = 384 the tiles of a last, partial round are shared by three CTAs each when that
// still fits one round: every one of the three forms the hidden activations, and accumulates
// and stores one 128-column third of Y (see the kernel).
//
// Warp roles (512 threads): warps 0 and 2 = weight TMA producers (warp 0 owns TMEM),
// warp 1 = UMMA issuer (warp 15 is idle), warps 3-6 = X row
// gather, warps 7-14 = epilogue (two warps per TMEM lane quarter).  Producer and issuer warps stay
// converged and elect one lane per instruction.  Every wait is bounded; on expiry the CTA raises SENTRY_STATUS_BIT_TIMEOUT
// and unwinds.
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "ffn_plan.cuh"
#include "tc_common.cuh"
#include "ptx/sm100.cuh"

namespace {

constexpr int kTileRows = 128;
constexpr int kBlockBytes = 128 * 128;   // 128 rows x 64 bf16: one X block, one hidden block
constexpr int kStageBytes = 2 * kBlockBytes;
constexpr int kStages = 3;
constexpr int kThreads = 512;
constexpr int kLoaderWarp0 = 3, kLoaderWarps = 4, kLoaderThreads = kLoaderWarps * 32;
constexpr int kEpiWarp0 = 7, kEpiWarps = 8;
constexpr int kTmemCols = 512;

// FP8: X, the weights and the hidden activations are e4m3 bytes (a 128-byte operand row then
// holds 128 elements instead of 64), the accumulators stay fp32, Y is stored as bf16.
template <int D, bool FP8 = false>
struct Cfg {
    static constexpr int EPB = FP8 ? 128 : 64;         // elements per 128-byte operand row
    static constexpr int CH = (D == 384) ? 128 : 256;  // kept channels per chunk
    static constexpr int CH16 = FP8 ? CH / 2 : CH;     // a chunk's width in the 16-bit units of the weight maps
    static constexpr int KB1 = D / EPB;                // X blocks per tile = K blocks of GEMM1
    static constexpr int H_COL0 = (D == 384) ? 384 : 256;  // TMEM column of the hidden accumulator
    static constexpr int NXS = (D == 128 || FP8) ? 4 : KB1;   // X block slots (two tiles' worth where they are few)
    static constexpr int NHS = CH / EPB;               // hidden blocks per chunk
    static constexpr int NBATCH = CH / 128;            // 64-column batches per epilogue warp
    static constexpr int SPG = (D == 384) ? 3 : KB1;   // weight stages per chunk of GEMM1 (= of GEMM2)
    static constexpr bool COLSPLIT = (D == 384);   // tail tiles shared by three CTAs, a third of Y each
    // FP8 with d_model = 384: one 128-channel hidden block, written by all eight epilogue warps, and two more
    // blocks that only stage Y on its way out (the hidden block is live while Y drains)
    static constexpr bool FP8_384 = FP8 && D == 384;
    static constexpr int NHS_ALLOC = FP8_384 ? 3 : NHS;
    static constexpr int OFF_H = NXS * kBlockBytes;
    static constexpr int OFF_W = OFF_H + NHS_ALLOC * kBlockBytes;
    static constexpr int OFF_MISC = OFF_W + kStages * kStageBytes;
    static constexpr int SMEM_BYTES = OFF_MISC + 2048 + 1024;  // + misc + alignment slack
    static_assert(SMEM_BYTES <= 232448, "shared memory over the per-CTA limit");
};

struct Misc {
    uint64_t w_full[kStages], w_empty[kStages];
    uint64_t x_full[8], x_empty[8];
    uint64_t h_full, h_tmem_empty;
    uint64_t hs_full[4], hs_empty[4];
    uint64_t y_full, y_empty;
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Misc) <= 2048, "misc block too large");

// ---- lean forms for the single-thread roles -------------------------------------------------
// A warp that walks a chain of dependent scalar instructions with shared-memory round trips in
// it (an mbarrier probe, a flag poll, a vote) advances at 8 to 15 cycles per instruction here,
// so what the producers and issuers execute per stage is counted in instructions: barrier
// addresses are one add from a base, descriptors are a 32-bit add and a register pair, all the
// probes of a stage are issued back to back and voted on once.
#define MISC_BAR(base, field) ((base) + (uint32_t)offsetof(Misc, field))
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // upper word of umma_smem_desc_sw128
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr) { return ((smem_addr >> 4) & 0x3fffu) | (1u << 16); }
// D (+)= A . B^T for one 128-byte K block = four 32-byte K steps (K = 16 16-bit or 32 8-bit elements);
// descriptors from their low words
#define SENTRY_MMA_KBLOCK(KIND)                                                                                       \
    asm volatile(                                                                                                     \
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"                                            \
        "setp.ne.b32 p, %5, 0;\n\t"                                                                                   \
        "mov.b64 da, {%1, %4};\n\tmov.b64 db, {%2, %4};\n\t"                                                          \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, p;\n\t"                                             \
        "setp.ne.b32 p, 1, 0;\n\t"                                                                                    \
        "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"              \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, p;\n\t"                                             \
        "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"              \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, p;\n\t"                                             \
        "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"              \
        "tcgen05.mma.cta_group::1.kind::" KIND " [%0], da, db, %3, p;\n\t}"                                            \
        :                                                                                                             \
        : "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(kDescHi), "r"(accumulate_first)                          \
        : "memory")
template <bool FP8>
__device__ __forceinline__ void mma_kblock(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                           uint32_t accumulate_first) {
    if constexpr (FP8) SENTRY_MMA_KBLOCK("f8f6f4");
    else SENTRY_MMA_KBLOCK("f16");
}
// Slow path of a stage's combined wait: the barriers one after the other, bounded (0 = none).
static __device__ __noinline__ bool wait_each_slow(uint32_t b0, uint32_t p0, uint32_t b1, uint32_t p1, uint32_t b2,
                                                   uint32_t p2, uint32_t b3, uint32_t p3, volatile int* abort_flag) {
    bool ok = ptx::mbar_wait(b0, p0, abort_flag);
    if (ok && b1 != 0u) ok = ptx::mbar_wait(b1, p1, abort_flag);
    if (ok && b2 != 0u) ok = ptx::mbar_wait(b2, p2, abort_flag);
    if (ok && b3 != 0u) ok = ptx::mbar_wait(b3, p3, abort_flag);
    return ok;
}

// End of a CTA: if any wait ran out, raise the status bit and give copies and UMMAs that may
// still be in flight time to land before shared memory and TMEM go away; then free the TMEM.
__device__ __forceinline__ void cta_teardown(volatile int* abort_flag, unsigned int* status, uint32_t tmem,
                                             uint32_t tmem_cols) {
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_TIMEOUT);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
        __syncthreads();
    }
    if ((threadIdx.x >> 5) == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, tmem_cols);
    }
}

// F16: X, W and Y are IEEE half instead of bf16.  FP8: X and the weights are e4m3 bytes with
// per-tensor scales, the hidden activations are requantised to e4m3 (gelu(acc * a_scale) * h_inv),
// Y = acc * y_scale is stored as bf16.
template <int D, bool F16, bool FP8 = false>
__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_w2_256,
              const __grid_constant__ CUtensorMap tm_w2_128, const __nv_bfloat16* __restrict__ X,
              __nv_bfloat16* __restrict__ Y, FfnPlan plan, int n_lists, int kc_pad,
              unsigned int* status, float a_scale, float h_inv, float y_scale) {
    using C = Cfg<D, FP8>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;   // 1024-byte aligned operand blocks
    uint8_t* smem = smem_raw + (base - raw_addr);
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);
    const uint32_t xs = base, hs = base + C::OFF_H, wsm = base + C::OFF_W;
    volatile int* abort_flag = &misc->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NC = kc_pad / C::CH;
    const int total_tiles = plan.tile_start[n_lists];
    // Column-split tail (d_model = 384, 16-bit and FP8 operands).  The tiles of the last, partial round leave most CTAs idle
    // (340 tiles on 148 CTAs: 44 in the third round).  When three times their number still fits
    // one round, each of them is taken by three CTAs: all three form the tile's hidden
    // activations, and each accumulates and stores one 128-column third of Y (GEMM2 of a third =
    // the N = 128 stage alone).  Nothing is exchanged; a third costs 4/6 of the tensor work of a
    // whole tile.  Virtual tile v < full_v is tile v; the others are (tile, third) pairs.  A CTA's
    // split tile, if it has one, is its last.
    int full_v = total_tiles, n_vt = total_tiles;
    if constexpr (C::COLSPLIT) {
        const int rem = total_tiles % (int)gridDim.x;
        if (rem > 0 && 3 * rem <= (int)gridDim.x) { full_v = total_tiles - rem; n_vt = full_v + 3 * rem; }
    }
    auto tile_of = [&](int v) { return v < full_v ? v : full_v + (v - full_v) / 3; };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->w_empty[s]), 1);
        }
        for (int s = 0; s < 8; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->x_full[s]), kLoaderWarps);
            ptx::mbar_init(ptx::smem_u32(&misc->x_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->h_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->h_tmem_empty), kEpiWarps);
        for (int b = 0; b < 4; ++b) {
            ptx::mbar_init(ptx::smem_u32(&misc->hs_full[b]), C::FP8_384 ? 8 : 4);   // one warp per TMEM lane quarter (FP8, 384: both halves)
            ptx::mbar_init(ptx::smem_u32(&misc->hs_empty[b]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->y_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->y_empty), kEpiWarps);
        misc->abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = misc->tmem_base;

    constexpr int SPG = C::SPG;
    const uint32_t mb = ptx::smem_u32(misc);
    const int my_tiles = (n_vt - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int last_v = (int)blockIdx.x + (my_tiles - 1) * (int)gridDim.x;
    const int my_third = (my_tiles > 0 && last_v >= full_v) ? (last_v - full_v) % 3 : -1;   // -1: no split tile
    const uint32_t n_chunks = (uint32_t)(my_tiles * NC);
    // Ring order: GEMM1 of chunk 0; then, per chunk q >= 1, GEMM1 of q and GEMM2 of q-1; at the
    // end GEMM2 of the last chunk.  Producers and issuers walk it as "group q = GEMM1(q), GEMM2(q-1)"
    // for q = 0 .. n_chunks, skipping the halves that do not exist; SPG stages per GEMM.
    if (warp == 0 || warp == 2) {
        // ----------------------------------------------------------- weight TMA producers
        // Producer p loads the stages with ring position n = p (mod 2).
        const uint32_t me = (warp == 0) ? 0u : 1u;
        if (elect_one()) {
            ptx::prefetch_tensormap(&tm_w1);
            ptx::prefetch_tensormap(&tm_w2_256);
            ptx::prefetch_tensormap(&tm_w2_128);
        }
        __syncwarp();
        // one stage = one 32 KB box, or two 16 KB boxes (x1 < 0: single box)
        auto stage = [&](uint32_t n, const CUtensorMap* tm, int x0, int x1, int y, uint32_t bytes = kStageBytes) -> bool {
            const uint32_t sl = n % kStages, use = n / kStages;
            const uint32_t we = MISC_BAR(mb, w_empty) + 8u * sl;
            if (!__all_sync(0xffffffffu, ptx::mbar_try_wait(we, (use & 1u) ^ 1u)) &&
                !__all_sync(0xffffffffu, ptx::mbar_wait_slow(we, (use & 1u) ^ 1u, abort_flag)))
                return false;
            if (elect_one()) {
                const uint32_t bar = MISC_BAR(mb, w_full) + 8u * sl;
                const uint32_t dst = wsm + sl * kStageBytes;
                ptx::mbar_arrive_expect_tx(bar, bytes);
                ptx::tma_load_2d(dst, tm, x0, y, bar);
                if (x1 >= 0) ptx::tma_load_2d(dst + kBlockBytes, tm, x1, y, bar);
            }
            __syncwarp();
            return true;
        };
        uint32_t n = 0;
        bool ok = true;
        int l_cur = 0, l_last = 0, c = 0;
        uint32_t ti = 0;
#pragma unroll 1
        for (uint32_t q = 0; q <= n_chunks && ok; ++q) {
            if (c == 0) {
                l_last = l_cur;
                if (q < n_chunks) {
                    int row0, n_rows;
                    ffn_tile_lookup(plan, n_lists, tile_of((int)blockIdx.x + (int)ti * (int)gridDim.x), kTileRows, l_cur, row0, n_rows);
                }
            }
            if (q < n_chunks) {
                const int y = l_cur * kc_pad + c * C::CH;
#pragma unroll
                for (int i = 0; i < SPG; ++i) {
                    if (ok && ((n + i) & 1u) == me) {
                        if constexpr (C::FP8_384) ok = stage(n + i, &tm_w1, 64 * i, -1, y, kBlockBytes);   // one 128-byte K block of 128 channels
                        else if constexpr (D == 384) ok = stage(n + i, &tm_w1, 128 * i, 128 * i + 64, y);
                        else ok = stage(n + i, &tm_w1, 64 * i, -1, y);
                    }
                }
                n += SPG;
            }
            if (q > 0) {
                const int pl = c ? l_cur : l_last, x = (c ? c - 1 : NC - 1) * C::CH16, y = pl * D;
                if constexpr (C::FP8_384) {
                    if (my_third >= 0 && (int)(c ? ti : ti - 1) == my_tiles - 1) {
                        // a third of Y: one 16 KB N = 128 stage
                        if (ok && (n & 1u) == me) ok = stage(n, &tm_w2_128, x, -1, y + 128 * my_third, kBlockBytes);
                        n += 1;
                    } else {
                        // the chunk is one K block: columns 0..255 of Y from an N = 256 stage, 256..383 from a 16 KB N = 128 stage
                        if (ok && (n & 1u) == me) ok = stage(n, &tm_w2_256, x, -1, y);
                        if (ok && ((n + 1) & 1u) == me) ok = stage(n + 1, &tm_w2_128, x, -1, y + 256, kBlockBytes);
                        n += 2;
                    }
                    if (++c == NC) { c = 0; ++ti; }
                    continue;
                }
                if (C::COLSPLIT && my_third >= 0 && (int)(c ? ti : ti - 1) == my_tiles - 1) {
                    // a third of Y: one N = 128 stage (both K blocks of the chunk)
                    if ((n & 1u) == me) ok = stage(n, &tm_w2_128, x, x + 64, y + 128 * my_third);
                    n += 1;
                    if (++c == NC) { c = 0; ++ti; }
                    continue;
                }
#pragma unroll
                for (int i = 0; i < SPG; ++i) {
                    if (ok && ((n + i) & 1u) == me) {
                        if constexpr (D == 256) {
                            ok = stage(n + i, &tm_w2_256, x + 64 * i, -1, y);
                        } else if constexpr (D == 128) {
                            ok = stage(n + i, &tm_w2_128, x + 128 * i, x + 128 * i + 64, y);
                        } else {
                            // columns 0..255 of Y from two N=256 stages, 256..383 from one N=128 stage
                            if (i < 2) ok = stage(n + i, &tm_w2_256, x + 64 * i, -1, y);
                            else ok = stage(n + i, &tm_w2_128, x, x + 64, y + 256);
                        }
                    }
                }
                n += SPG;
            }
            if (++c == NC) { c = 0; ++ti; }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------- UMMA issuer
        // One warp walks the schedule of weight stages; for every stage it probes the barriers
        // the stage needs (weights landed, operand blocks written, accumulator released), and
        // one elected lane issues the stage's UMMAs and commits.  ALL UMMAs come from one
        // thread: the tensor pipe runs the instructions of one thread in issue order, but
        // nothing orders the instructions of two threads, and accumulators fed alternately by
        // two issuing warps were summed in an order that changed from run to run (results
        // differed in the last bit).  A second warp that did the waiting and handed the stage
        // number over through shared memory measured slower than the issuer waiting itself.
        // (kind::f8f6f4 with both operand formats e4m3 has the same descriptor bits as kind::f16 with fp16 operands:
        // format code 0 for A and B, fp32 accumulator)
        constexpr uint32_t idesc256 = (F16 || FP8) ? ptx::umma_idesc_f16(128, 256) : ptx::umma_idesc_bf16(128, 256);
        constexpr uint32_t idesc128 = (F16 || FP8) ? ptx::umma_idesc_f16(128, 128) : ptx::umma_idesc_bf16(128, 128);
        constexpr uint32_t kBlkLo = kBlockBytes >> 4, kStageLo = kStageBytes >> 4;
        const uint32_t tm_h = tmem + C::H_COL0;
        const uint32_t xs_lo = desc_lo(xs), hs_lo = desc_lo(hs), w_lo = desc_lo(wsm);
        // One stage.  wb*: barriers to wait on besides the weights (0 = none), cb*: barriers to
        // commit to besides w_empty (0 = none); a_lo1 != 0: the stage holds two K blocks.
        auto stage = [&](uint32_t n, uint32_t d_tm, uint32_t a_lo0, uint32_t a_lo1, uint32_t idesc, bool overwrite,
                         uint32_t wb0, uint32_t wp0, uint32_t wb1, uint32_t wp1, uint32_t wb2, uint32_t wp2,
                         bool /*writes TMEM others read: fenced in every case*/, uint32_t cb0, uint32_t cb1,
                         uint32_t cb2) -> bool {
            const uint32_t sl = n % kStages, ph = (n / kStages) & 1u;
            {
                const uint32_t wf = MISC_BAR(mb, w_full) + 8u * sl;
                bool p = ptx::mbar_try_wait(wf, ph);
                if (wb0 != 0u) p &= ptx::mbar_try_wait(wb0, wp0);
                if (wb1 != 0u) p &= ptx::mbar_try_wait(wb1, wp1);
                if (wb2 != 0u) p &= ptx::mbar_try_wait(wb2, wp2);
                if (!__all_sync(0xffffffffu, p) &&
                    !__all_sync(0xffffffffu, wait_each_slow(wf, ph, wb0, wp0, wb1, wp1, wb2, wp2, abort_flag)))
                    return false;
            }
            ptx::tc_fence_after_sync();   // orders the UMMAs after the epilogue's TMEM reads and operand writes
            if (elect_one()) {
                const uint32_t b_lo = w_lo + sl * kStageLo;
                mma_kblock<FP8>(d_tm, a_lo0, b_lo, idesc, overwrite ? 0u : 1u);
                if (a_lo1 != 0u) mma_kblock<FP8>(d_tm, a_lo1, b_lo + kBlkLo, idesc, 1u);
                if (cb0 != 0u) ptx::umma_commit(cb0);
                if (cb1 != 0u) ptx::umma_commit(cb1);
                ptx::umma_commit(MISC_BAR(mb, w_empty) + 8u * sl);
                if (cb2 != 0u) ptx::umma_commit(cb2);
            }
            __syncwarp();
            return true;
        };
        uint32_t n = 0, ti = 0;
        bool ok = true;
        int c = 0;
#pragma unroll 1
        for (uint32_t q = 0; q <= n_chunks && ok; ++q) {
            if (q < n_chunks) {
                // GEMM1 of chunk q = chunk c of local tile ti:  H = X . W1c_chunk^T
                const bool last = (c == NC - 1), first = (c == 0);
                const uint32_t hp = (q & 1u) ^ 1u;
#pragma unroll
                for (int i = 0; i < SPG; ++i) {
                    if (!ok) continue;
                    const uint32_t he = (i == 0) ? MISC_BAR(mb, h_tmem_empty) : 0u;
                    const uint32_t hf = (i == SPG - 1) ? MISC_BAR(mb, h_full) : 0u;
                    if constexpr (D == 384 && !FP8) {
                        const uint32_t s0 = 2 * i, s1 = 2 * i + 1;   // X slots (NXS = KB1 = 6)
                        ok = stage(n + i, tm_h, xs_lo + s0 * kBlkLo, xs_lo + s1 * kBlkLo, idesc128, i == 0,
                                   first ? MISC_BAR(mb, x_full) + 8u * s0 : 0u, ti & 1u,
                                   first ? MISC_BAR(mb, x_full) + 8u * s1 : 0u, ti & 1u, he, hp, i == 0,
                                   last ? MISC_BAR(mb, x_empty) + 8u * s0 : 0u,
                                   last ? MISC_BAR(mb, x_empty) + 8u * s1 : 0u, hf);
                    } else {
                        const uint32_t gx = ti * C::KB1 + i, slot = gx % C::NXS;
                        ok = stage(n + i, tm_h, xs_lo + slot * kBlkLo, 0u, C::CH == 256 ? idesc256 : idesc128, i == 0,
                                   first ? MISC_BAR(mb, x_full) + 8u * slot : 0u, (gx / C::NXS) & 1u, 0u, 0u, he, hp,
                                   i == 0, last ? MISC_BAR(mb, x_empty) + 8u * slot : 0u, 0u, hf);
                    }
                }
                n += SPG;
            }
            if (q > 0 && ok) {
                // GEMM2 of chunk q-1 = chunk pc of local tile pti:  Y (+)= gelu(H) . W2c_chunk
                const int pc = c ? c - 1 : NC - 1;
                const uint32_t pti = c ? ti : ti - 1, gp = (q - 1) & 1u;
                const bool first = (pc == 0), last = (pc == NC - 1);
                const uint32_t ye = first ? MISC_BAR(mb, y_empty) : 0u, yp = (pti & 1u) ^ 1u;
                const uint32_t yf = last ? MISC_BAR(mb, y_full) : 0u;
                if constexpr (C::FP8_384) {
                    if (my_third >= 0 && (int)pti == my_tiles - 1) {
                        ok = stage(n, tmem + 128u * (uint32_t)my_third, hs_lo, 0u, idesc128, first, MISC_BAR(mb, hs_full), gp,
                                   0u, 0u, ye, yp, first, MISC_BAR(mb, hs_empty), 0u, yf);
                        n += 1;
                    } else {
                        ok = stage(n, tmem, hs_lo, 0u, idesc256, first, MISC_BAR(mb, hs_full), gp, 0u, 0u, ye, yp, first, 0u, 0u, 0u);
                        if (ok)
                            ok = stage(n + 1, tmem + 256u, hs_lo, 0u, idesc128, first, 0u, 0u, 0u, 0u, 0u, 0u, first,
                                       MISC_BAR(mb, hs_empty), 0u, yf);
                        n += 2;
                    }
                    if (++c == NC) { c = 0; ++ti; }
                    continue;
                }
                if (C::COLSPLIT && my_third >= 0 && (int)pti == my_tiles - 1) {
                    ok = stage(n, tmem + 128u * (uint32_t)my_third, hs_lo, hs_lo + kBlkLo, idesc128, first,
                               MISC_BAR(mb, hs_full), gp, MISC_BAR(mb, hs_full) + 8u, gp, ye, yp, first,
                               MISC_BAR(mb, hs_empty), MISC_BAR(mb, hs_empty) + 8u, yf);
                    n += 1;
                    if (++c == NC) { c = 0; ++ti; }
                    continue;
                }
#pragma unroll
                for (int i = 0; i < SPG; ++i) {
                    if (!ok) continue;
                    if constexpr (D == 256) {
                        ok = stage(n + i, tmem, hs_lo + i * kBlkLo, 0u, idesc256, first && i == 0,
                                   MISC_BAR(mb, hs_full) + 8u * i, gp, 0u, 0u, i == 0 ? ye : 0u, yp, first && i == 0,
                                   MISC_BAR(mb, hs_empty) + 8u * i, 0u, i == SPG - 1 ? yf : 0u);
                    } else if constexpr (D == 128) {
                        const int k0 = 2 * i, k1 = 2 * i + 1;
                        ok = stage(n + i, tmem, hs_lo + k0 * kBlkLo, hs_lo + k1 * kBlkLo, idesc128, first && i == 0,
                                   MISC_BAR(mb, hs_full) + 8u * k0, gp, MISC_BAR(mb, hs_full) + 8u * k1, gp,
                                   i == 0 ? ye : 0u, yp, first && i == 0, MISC_BAR(mb, hs_empty) + 8u * k0,
                                   MISC_BAR(mb, hs_empty) + 8u * k1, i == SPG - 1 ? yf : 0u);
                    } else {
                        // columns 0..255 of Y from two N=256 stages, columns 256..383 from one N=128
                        // stage that needs both hidden blocks (and, on the first chunk, Y's release)
                        if (i < 2) {
                            ok = stage(n + i, tmem, hs_lo + i * kBlkLo, 0u, idesc256, first && i == 0,
                                       MISC_BAR(mb, hs_full) + 8u * i, gp, 0u, 0u, i == 0 ? ye : 0u, yp,
                                       first && i == 0, 0u, 0u, 0u);
                        } else {
                            ok = stage(n + i, tmem + 256, hs_lo, hs_lo + kBlkLo, idesc128, first,
                                       MISC_BAR(mb, hs_full), gp, MISC_BAR(mb, hs_full) + 8u, gp, ye, yp, first,
                                       MISC_BAR(mb, hs_empty), MISC_BAR(mb, hs_empty) + 8u, yf);
                        }
                    }
                }
                n += SPG;
            }
            if (++c == NC) { c = 0; ++ti; }
        }
    } else if (warp >= kLoaderWarp0 && warp < kEpiWarp0) {
        // ------------------------------------------------------------------ X row gather
        // Thread -> 8 (row, 16-byte chunk) pairs of every 128 x 64 block.  Up to three blocks
        // are in flight per thread; a block is published (x_full, one arrival per warp) once
        // the copies of all lanes have landed.
        const int tl = threadIdx.x - kLoaderWarp0 * 32;
        uint32_t gx = 0, published = 0;   // blocks issued / published by this warp
        bool ok = true;
        auto publish_oldest = [&]() {
            cp_async_wait_pending((int)(gx - published) - 1);
            ptx::fence_proxy_async_smem();
            warp_arrive(&misc->x_full[published % C::NXS]);
            ++published;
        };
        for (int vt = blockIdx.x; vt < n_vt && ok; vt += gridDim.x) {
            int l, row0, n_rows;
            ffn_tile_lookup(plan, n_lists, tile_of(vt), kTileRows, l, row0, n_rows);
            int32_t rows[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int r = (tl + j * kLoaderThreads) >> 3;
                rows[j] = r < n_rows ? plan.rowidx[row0 + r] : -1;
            }
            for (int kb = 0; kb < C::KB1 && ok; ++kb) {
                const uint32_t slot = gx % C::NXS, use = gx / C::NXS;
                uint64_t* bar = &misc->x_empty[slot];
                // never block on a slot while holding unpublished blocks the issuer may need
                while (gx > published &&
                       !__all_sync(0xffffffffu, ptx::mbar_test_wait(ptx::smem_u32(bar), (use & 1u) ^ 1u)))
                    publish_oldest();
                if (!warp_wait(bar, (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int idx = tl + j * kLoaderThreads;
                    const int r = idx >> 3, ci = idx & 7;
                    const uint32_t dst = xs + slot * kBlockBytes + r * 128 + ((ci ^ (r & 7)) << 4);
                    if (rows[j] >= 0) {
                        if constexpr (FP8)
                            ptx::cp_async_16(dst, reinterpret_cast<const uint8_t*>(X) + (size_t)rows[j] * D + kb * 128 + ci * 16);
                        else
                            ptx::cp_async_16(dst, X + (size_t)rows[j] * D + kb * 64 + ci * 8);
                    } else {
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
                    }
                }
                ptx::cp_async_commit();
                ++gx;
                if (gx - published == 3) publish_oldest();
            }
        }
        while (ok && gx > published) publish_oldest();
        ptx::cp_async_wait_all();
    } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
        // ---------------------------------------------------------------------- epilogue
        const int ew = warp - kEpiWarp0;
        const int quarter = warp & 3, half = ew >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        uint32_t g = 0, ti = 0;
        bool ok = true;
        int32_t my_row = -1, prev_row = -1;
        // Y of a finished tile: TMEM -> bf16 -> global, then hand the accumulator back.  Each
        // lane holds one row; 64 columns at a time go through this warp's 4 KB piece of the
        // hidden-block buffer (free while Y is complete and this warp has not yet written its
        // next hidden block there) so that the global stores cover whole 128-byte row segments.
        constexpr int kDrainBlk = C::NBATCH - 1;
        // (FP8: a warp writes one 128-channel hidden block, rows of its own quarter: that piece)
        const uint32_t stg = C::FP8_384 ? hs + (uint32_t)(1 + half) * kBlockBytes + (uint32_t)quarter * 4096u
                           : FP8 ? hs + (uint32_t)half * kBlockBytes + (uint32_t)quarter * 4096u
                                 : hs + (uint32_t)(half * C::NBATCH + kDrainBlk) * kBlockBytes + (uint32_t)quarter * 4096u;
        auto drain_y = [&](uint32_t t_idx, int32_t grow, int third) {
            if (!warp_wait(&misc->y_full, t_idx & 1u, abort_flag)) { ok = false; return; }
            ptx::tc_fence_after_sync();
            // 64 columns per pass: two TMEM loads and one wait, bf16 rows through the staging
            // piece, then whole 128-byte row segments to global memory.  The registers a TMEM
            // load writes are not named again before its wait.
            // a whole tile: this half's D/2 columns in passes of 64; a third: 64 of its 128 columns
            const int NP = third < 0 ? D / 128 : 1;
            const int cbase = third < 0 ? half * (D / 2) : third * 128 + half * 64;
            const int ch = lane & 7;
            int32_t grs[8];
#pragma unroll
            for (int step = 0; step < 8; ++step) grs[step] = __shfl_sync(0xffffffffu, grow, step * 4 + (lane >> 3));
            __nv_bfloat16* ycol = Y + cbase + ch * 8;
#pragma unroll 1
            for (int pass = 0; pass < NP; ++pass) {
                uint32_t ra[32], rb[32];
                const int col0 = cbase + pass * 64;
                ptx::tmem_ld_32x32(lane_base + col0, ra);
                ptx::tmem_ld_32x32(lane_base + col0 + 32, rb);
                ptx::tmem_ld_wait();
                if constexpr (FP8) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        ra[i] = __float_as_uint(__uint_as_float(ra[i]) * y_scale);
                        rb[i] = __float_as_uint(__uint_as_float(rb[i]) * y_scale);
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + ((i ^ (lane & 7)) << 4)),
                                 "r"(pack_16x2<F16>(__uint_as_float(ra[8 * i]), __uint_as_float(ra[8 * i + 1]))),
                                 "r"(pack_16x2<F16>(__uint_as_float(ra[8 * i + 2]), __uint_as_float(ra[8 * i + 3]))),
                                 "r"(pack_16x2<F16>(__uint_as_float(ra[8 * i + 4]), __uint_as_float(ra[8 * i + 5]))),
                                 "r"(pack_16x2<F16>(__uint_as_float(ra[8 * i + 6]), __uint_as_float(ra[8 * i + 7])))
                                 : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((4 + i) ^ (lane & 7)) << 4)),
                                 "r"(pack_16x2<F16>(__uint_as_float(rb[8 * i]), __uint_as_float(rb[8 * i + 1]))),
                                 "r"(pack_16x2<F16>(__uint_as_float(rb[8 * i + 2]), __uint_as_float(rb[8 * i + 3]))),
                                 "r"(pack_16x2<F16>(__uint_as_float(rb[8 * i + 4]), __uint_as_float(rb[8 * i + 5]))),
                                 "r"(pack_16x2<F16>(__uint_as_float(rb[8 * i + 6]), __uint_as_float(rb[8 * i + 7])))
                                 : "memory");
                }
                __syncwarp();
#pragma unroll
                for (int step = 0; step < 8; ++step) {
                    const int rr = step * 4 + (lane >> 3);
                    uint4 v;
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                 : "r"(stg + rr * 128 + ((ch ^ (rr & 7)) << 4)));
                    if (grs[step] >= 0) *reinterpret_cast<uint4*>(ycol + (size_t)grs[step] * D + pass * 64) = v;
                }
                __syncwarp();
            }
            ptx::tc_fence_before_sync();
            warp_arrive(&misc->y_empty);
        };
        for (int vt = blockIdx.x; vt < n_vt && ok; vt += gridDim.x, ++ti) {
            int l, row0, n_rows;
            ffn_tile_lookup(plan, n_lists, tile_of(vt), kTileRows, l, row0, n_rows);
            prev_row = my_row;
            my_row = row < n_rows ? (plan.rowout ? plan.rowout : plan.rowidx)[row0 + row] : -1;
            for (int c = 0; c < NC && ok; ++c, ++g) {
                if (!warp_wait(&misc->h_full, g & 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int j = 0; j < C::NBATCH && ok; ++j) {
                    // 32 rows x 64 columns of the hidden accumulator -> registers
                    const int blk = half * C::NBATCH + j;        // hidden block = 64 channels (FP8: column batch)
                    // Y of the previous tile is complete about now (its last GEMM2 was queued right
                    // after this tile's first GEMM1): store it before this warp's last batch of the
                    // chunk is loaded, while no accumulator values are held in registers
                    // (FP8: before the first batch -- the staging piece is the block this warp is about to write)
                    if (j == (FP8 ? 0 : C::NBATCH - 1) && c == 0 && ti > 0) {
                        drain_y((uint32_t)(ti - 1), prev_row, -1);   // a split tile is the last one: never drained here
                        if (!ok) break;
                    }
                    uint32_t h0[32], h1[32];
                    const uint32_t tcol = lane_base + C::H_COL0 + blk * 64;
                    ptx::tmem_ld_32x32(tcol, h0);
                    ptx::tmem_ld_32x32(tcol + 32, h1);
                    ptx::tmem_ld_wait();
                    if (j == C::NBATCH - 1) {
                        // the accumulator is in registers: GEMM1 of the next chunk may start
                        ptx::tc_fence_before_sync();
                        warp_arrive(&misc->h_tmem_empty);
                    }
                    if constexpr (FP8) {
                        // 64 columns -> 64 e4m3 bytes = chunks 4j .. 4j+3 of this row of hidden block `half`
                        uint32_t p8[16];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            p8[i] = gelu_pack_e4m3x4(__uint_as_float(h0[4 * i]) * a_scale, __uint_as_float(h0[4 * i + 1]) * a_scale,
                                                     __uint_as_float(h0[4 * i + 2]) * a_scale, __uint_as_float(h0[4 * i + 3]) * a_scale, h_inv);
                            p8[8 + i] = gelu_pack_e4m3x4(__uint_as_float(h1[4 * i]) * a_scale, __uint_as_float(h1[4 * i + 1]) * a_scale,
                                                         __uint_as_float(h1[4 * i + 2]) * a_scale, __uint_as_float(h1[4 * i + 3]) * a_scale, h_inv);
                        }
                        // (d_model 384: one hidden block for the chunk, this warp's 64 channels are bytes 64 half .. of a row)
                        constexpr bool ONE = C::FP8_384;
                        const int hb = ONE ? 0 : half, cb = ONE ? 4 * half : 4 * j;
                        if (j == 0 && !warp_wait(&misc->hs_empty[hb], (g & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t hrow8 = hs + hb * kBlockBytes + row * 128;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t dst = hrow8 + (((cb + i) ^ (row & 7)) << 4);
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(p8[4 * i]),
                                         "r"(p8[4 * i + 1]), "r"(p8[4 * i + 2]), "r"(p8[4 * i + 3])
                                         : "memory");
                        }
                        if (j == C::NBATCH - 1) {
                            ptx::fence_proxy_async_smem();
                            warp_arrive(&misc->hs_full[hb]);
                        }
                        continue;
                    }
                    uint32_t pk[32];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        pk[i] = gelu_pack_16x2<F16>(__uint_as_float(h0[2 * i]), __uint_as_float(h0[2 * i + 1]));
                        pk[16 + i] = gelu_pack_16x2<F16>(__uint_as_float(h1[2 * i]), __uint_as_float(h1[2 * i + 1]));
                    }
                    if (!warp_wait(&misc->hs_empty[blk], (g & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t hrow = hs + blk * kBlockBytes + row * 128;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t dst = hrow + ((i ^ (row & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * i]),
                                     "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                                     : "memory");
                    }
                    ptx::fence_proxy_async_smem();
                    warp_arrive(&misc->hs_full[blk]);
                }
            }
        }
        if (ok && ti > 0) drain_y(ti - 1, my_row, my_third);
    }

    cta_teardown(abort_flag, status, tmem, kTmemCols);
}

// One CTA that waits, through the same bounded wait as the kernels above, on a barrier nobody
// ever arrives on, and then unwinds through the same teardown (status bit, grace period, TMEM
// release).  It exists so that a test can watch a wait run out without hanging anything.
__global__ void __launch_bounds__(128, 1) wait_expiry_selftest_kernel(long long limit_cycles, unsigned int* status) {
    __shared__ uint64_t never;
    __shared__ uint32_t tmem_base;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&never), 1);
        abort_word = 0;
        ptx::fence_barrier_init();
    }
    if ((threadIdx.x >> 5) == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base), 32);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = tmem_base;
    // warp 1 waits with the limit under test; the other warps wait with the default limit and
    // must be released by the abort flag that warp 1 raises
    const long long limit = (threadIdx.x >> 5) == 1 ? limit_cycles : ptx::kWaitLimitCycles;
    (void)ptx::mbar_wait(ptx::smem_u32(&never), 0u, abort_flag, limit);
    cta_teardown(abort_flag, status, tmem, 32);
}

template <int D, bool F16>
int launch_d(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c, int kc_pad,
             int max_tiles, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    CUtensorMap m1, m2a, m2b;
    const uint64_t r1 = (uint64_t)d.n_lists * kc_pad, r2 = (uint64_t)d.n_lists * D;
    if (!make_weight_map(&m1, w1c, r1, D, Cfg<D>::CH == 256 ? 256 : 128)) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2a, w2c, r2, kc_pad, D >= 256 ? 256 : 128)) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2b, w2c, r2, kc_pad, 128)) return SENTRY_ERR_CUDA;
    auto kern = ffn_tc_kernel<D, F16>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::SMEM_BYTES));
    int grid = max_tiles < ctx->sm_count ? max_tiles : ctx->sm_count;
    if (grid < 1) grid = 1;
    LaunchScope ls(ctx, KS_FFN_MAIN, st);
    kern<<<grid, kThreads, Cfg<D>::SMEM_BYTES, st>>>(m1, m2a, m2b, (const __nv_bfloat16*)a.X,
                                                      (__nv_bfloat16*)a.Y, plan, d.n_lists, kc_pad, a.status, 1.f, 1.f, 1.f);
    return SENTRY_OK;
}

// FP8 (e4m3 bytes): the weight maps describe the same bytes as 16-bit elements, two e4m3 each.
template <int D>
int launch_fp8(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c, int kc_pad,
               int max_tiles, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    CUtensorMap m1, m2a, m2b;
    const uint64_t r1 = (uint64_t)d.n_lists * kc_pad, r2 = (uint64_t)d.n_lists * D;
    if (!make_weight_map(&m1, w1c, r1, D / 2, Cfg<D, true>::CH == 256 ? 256 : 128)) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2a, w2c, r2, kc_pad / 2, 256)) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2b, w2c, r2, kc_pad / 2, 128)) return SENTRY_ERR_CUDA;
    auto kern = ffn_tc_kernel<D, false, true>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D, true>::SMEM_BYTES));
    int grid = max_tiles < ctx->sm_count ? max_tiles : ctx->sm_count;
    if (grid < 1) grid = 1;
    LaunchScope ls(ctx, KS_FFN_MAIN, st);
    kern<<<grid, kThreads, Cfg<D, true>::SMEM_BYTES, st>>>(m1, m2a, m2b, (const __nv_bfloat16*)a.X, (__nv_bfloat16*)a.Y,
                                                           plan, d.n_lists, kc_pad, a.status, a.fp8_a_scale,
                                                           a.fp8_h_inv, a.fp8_y_scale);
    return SENTRY_OK;
}

}  // namespace

bool ffn_tc_fp8_supported(const sentry_ffn_desc& d) {
    return d.dtype == SENTRY_FP8_E4M3 && (d.D == 128 || d.D == 256 || d.D == 384);
}

bool ffn_tc_supported(const sentry_ffn_desc& d) {
    if (d.dtype == SENTRY_FP8_E4M3) return d.D == 128 || d.D == 256 || d.D == 384;
    return (d.dtype == SENTRY_BF16 || d.dtype == SENTRY_F16) && (d.D == 128 || d.D == 256 || d.D == 384);
}

// kept channels are padded with zero columns / rows to a whole number of chunks
int ffn_tc_kc_pad(int D, int k_c) {
    const int ch = (D == 384) ? 128 : 256;
    return (k_c + ch - 1) / ch * ch;
}

int launch_wait_expiry_selftest(sentry_ctx* ctx, long long limit_cycles, cudaStream_t st) {
    wait_expiry_selftest_kernel<<<1, 128, 0, st>>>(limit_cycles, ctx->d_status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

int launch_ffn_tc(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c,
                  int kc_pad, int max_tiles, cudaStream_t st) {
    int rc;
    // the two 16-bit types share everything but the operand format of the UMMAs and the roundings
    // (X, Y and the weight tiles are moved as 16-bit words)
    if (a.d.dtype == SENTRY_FP8_E4M3) {
        if (!ffn_tc_fp8_supported(a.d)) return SENTRY_ERR_UNSUPPORTED;
        rc = a.d.D == 256 ? launch_fp8<256>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st)
             : a.d.D == 384 ? launch_fp8<384>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st)
                            : launch_fp8<128>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st);
        if (rc != SENTRY_OK) return rc;
        SENTRY_CUDA_TRY(cudaGetLastError());
        return SENTRY_OK;
    }
    const bool f16 = a.d.dtype == SENTRY_F16;
    switch (a.d.D) {
        case 128: rc = f16 ? launch_d<128, true>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st)
                           : launch_d<128, false>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st); break;
        case 256: rc = f16 ? launch_d<256, true>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st)
                           : launch_d<256, false>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st); break;
        case 384: rc = f16 ? launch_d<384, true>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st)
                           : launch_d<384, false>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st); break;
        default: return SENTRY_ERR_UNSUPPORTED;
    }
    if (rc != SENTRY_OK) return rc;
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

// Channel-compacted FFN on pairs of CTAs (Section 4.6):
//   Y = gelu(X . W1[:, N]) . W2[N, :]   for the present rows of every sample.
//
// Same computation and the same per-CTA pipeline as ffn_tc.cu (persistent CTAs, 128 rows per
// CTA, chunks of CH kept channels, GEMM1 -> GELU epilogue -> GEMM2 with both accumulators in
// TMEM), but the two CTAs of a cluster work on one tile of 256 rows and run every UMMA
// together (cta_group::2, M = 256): each CTA gathers its own 128 rows of X, keeps its own half
// of the hidden tile and of Y, and fetches only ONE HALF of every weight block; the tensor
// cores of both SMs read both halves.  A 32 KB ring slot per CTA therefore feeds 1024
// tensor-pipe cycles instead of 512, so the fixed cost of a slot hand-over (barrier waits, copy
// issue, commits by single threads) is spread over twice the arithmetic, and the weight
// traffic from L2 into shared memory is halved.
//
// Who talks to whom.  All UMMAs are issued by one thread of the even CTA of the pair (the
// leader).  Barriers the issuer waits on (weights landed, X block
// landed, hidden block written, accumulators drained) live in the leader's shared memory and
// count arrivals from BOTH CTAs: the peer arrives remotely, its TMA copies credit their bytes
// to the leader's barrier.  Barriers the issuer signals (ring slot free, X slot free, hidden
// accumulator ready, hidden slot free, Y ready) exist in both CTAs and are signalled by one
// multicast commit.  No multicast copies anywhere: every CTA loads its own operands.
//
// Warp roles per CTA (512 threads): warps 0 and 2 = weight TMA producers (warp 0 owns TMEM),
// warp 1 = UMMA issuer (leader only; idle in the peer; warp 15 is idle), warps 3-6 = X row gather,
// warps 7-14 = epilogue.  Every wait is bounded; on expiry the CTA raises
// SENTRY_STATUS_BIT_TIMEOUT and unwinds, and the pair leaves together.
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "ffn_plan.cuh"
#include "ffn_tc_common.cuh"
#include "ptx/sm100.cuh"

namespace {

constexpr int kTileRows = 128;           // rows per CTA
constexpr int kPairRows = 2 * kTileRows; // rows per tile of the plan
constexpr int kBlockBytes = 128 * 128;   // 128 rows x 64 bf16: one X block, one hidden block
constexpr int kSlotBytes = 2 * kBlockBytes;
constexpr int kStages = 3;
constexpr int kThreads = 512;
constexpr int kLoaderWarp0 = 3, kLoaderWarps = 4, kLoaderThreads = kLoaderWarps * 32;
constexpr int kEpiWarp0 = 7, kEpiWarps = 8;
constexpr int kTmemCols = 512;
constexpr int kMaxKb = 4;                // K blocks (64 wide) per ring slot at most

template <int D>
struct Cfg {
    static constexpr int CH = (D == 384) ? 128 : 256;  // kept channels per chunk
    static constexpr int KB1 = D / 64;                 // X blocks per tile = K blocks of GEMM1
    static constexpr int H_COL0 = (D == 384) ? 384 : 256;  // TMEM column of the hidden accumulator
    static constexpr int NXS = (D == 128) ? 4 : KB1;   // X block slots (D = 128: two tiles' worth)
    static constexpr int NHS = CH / 64;                // hidden blocks per chunk
    static constexpr int NBATCH = CH / 128;            // 64-column batches per epilogue warp
    static constexpr int SPG = (D == 128) ? 1 : 2;     // ring slots per GEMM of a chunk
    static constexpr int OFF_H = NXS * kBlockBytes;
    static constexpr int OFF_W = OFF_H + NHS * kBlockBytes;
    static constexpr int OFF_MISC = OFF_W + kStages * kSlotBytes;
    static constexpr int SMEM_BYTES = OFF_MISC + 2048 + 1024;
    static_assert(SMEM_BYTES <= 232448, "shared memory over the per-CTA limit");
};

// What one ring slot holds, per CTA: `nkb` K blocks of `rows` weight rows x 64, consecutive.
//   GEMM1 (B = W1c rows = kept channels of the chunk, this CTA's half of them):
//     D = 128: 128 rows x 2 blocks      D = 256: 128 rows x 2 blocks (slot i: K blocks 2i, 2i+1)
//     D = 384:  64 rows x 3 blocks (slot i: K blocks 3i .. 3i+2)
//   GEMM2 (B = W2c rows = output columns, this CTA's half of them):
//     D = 128:  64 rows x 4 blocks      D = 256: 128 rows x 2 blocks (slot i: hidden blocks 2i, 2i+1)
//     D = 384: slot 0 = 128 rows x 2 blocks (Y columns 0..255), slot 1 = 64 rows x 2 blocks (256..383)
template <int D>
struct SlotShape {
    __host__ __device__ static constexpr int g1_rows() { return D == 384 ? 64 : 128; }
    __host__ __device__ static constexpr int g1_nkb() { return D == 384 ? 3 : 2; }
    __host__ __device__ static constexpr int g2_rows(int i) { return D == 128 ? 64 : (D == 256 ? 128 : (i == 0 ? 128 : 64)); }
    __host__ __device__ static constexpr int g2_nkb() { return D == 128 ? 4 : 2; }
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

#define MISC_BAR(base, field) ((base) + (uint32_t)offsetof(Misc, field))
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // upper word of the 128-byte-swizzle descriptor
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr) { return ((smem_addr >> 4) & 0x3fffu) | (1u << 16); }

// D (+)= A . B^T for one 64-wide K block = four K=16 steps, issued for the CTA pair.
__device__ __forceinline__ void mma_kblock_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                                uint32_t accumulate_first) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %4};\n\tmov.b64 db, {%2, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t"
        "setp.ne.b32 p, 1, 0;\n\t"
        "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\tmov.b64 da, {ta, %4};\n\tmov.b64 db, {tb, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
        :
        : "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(kDescHi), "r"(accumulate_first)
        : "memory");
}

// Bounded wait on a barrier whose arrivals may come from the peer CTA.
static __device__ __noinline__ bool wait_cluster_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (ptx::mbar_try_wait_cluster(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > ptx::kWaitLimitCycles) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}
// One arrival for the whole warp on the barrier at this offset in the leader CTA.
__device__ __forceinline__ void warp_arrive_leader(uint64_t* bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) {
        if (ptx::cluster_ctarank() == 0) ptx::mbar_arrive(ptx::smem_u32(bar));
        else ptx::mbar_arrive_cluster(ptx::smem_u32(bar), 0u);
    }
}

// What the issuer does for one ring slot.
struct SlotWork {
    uint32_t d_tm, idesc, b_blk_lo;     // accumulator, instruction descriptor, bytes >> 4 between the slot's K blocks
    uint32_t a_lo[kMaxKb];              // A operand (X slot or hidden block) of every K block
    int nkb;
    bool overwrite;                     // first K block starts the accumulator afresh
    uint32_t wb[kMaxKb + 1], wp[kMaxKb + 1];   // barriers to wait on besides the weights (0 = none)
    uint32_t cb[kMaxKb + 1];            // barriers to commit to besides the ring slot (0 = none)
};

template <int D>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
ffn_tc_pair_kernel(const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_w2_128,
                   const __grid_constant__ CUtensorMap tm_w2_64, const __nv_bfloat16* __restrict__ X,
                   __nv_bfloat16* __restrict__ Y, FfnPlan plan, int n_lists, int kc_pad,
                   unsigned int* status) {
    using C = Cfg<D>;
    using SS = SlotShape<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;   // same offset in both CTAs of the pair
    uint8_t* smem = smem_raw + (base - raw_addr);
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);
    const uint32_t xs = base, hs = base + C::OFF_H, wsm = base + C::OFF_W;
    volatile int* abort_flag = &misc->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();        // 0 = leader
    const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);
    const int NC = kc_pad / C::CH;
    const int total_tiles = plan.tile_start[n_lists];

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->w_empty[s]), 1);
        }
        for (int s = 0; s < 8; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->x_full[s]), 2 * kLoaderWarps);
            ptx::mbar_init(ptx::smem_u32(&misc->x_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->h_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->h_tmem_empty), 2 * kEpiWarps);
        for (int b = 0; b < 4; ++b) {
            ptx::mbar_init(ptx::smem_u32(&misc->hs_full[b]), 2 * 4);   // one warp per TMEM lane quarter, both CTAs
            ptx::mbar_init(ptx::smem_u32(&misc->hs_empty[b]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->y_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->y_empty), 2 * kEpiWarps);
        misc->abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc_pair(ptx::smem_u32(&misc->tmem_base), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync_all();     // both CTAs' barriers exist before anyone arrives remotely
    ptx::tc_fence_after_sync();
    const uint32_t tmem = misc->tmem_base;

    constexpr int SPG = C::SPG;
    const uint32_t mb = ptx::smem_u32(misc);
    const int my_tiles = pair < total_tiles ? (total_tiles - pair + n_pairs - 1) / n_pairs : 0;
    const uint32_t n_chunks = (uint32_t)(my_tiles * NC);
    // Ring order as in the single-CTA kernel: "group q = GEMM1(chunk q), GEMM2(chunk q-1)" for
    // q = 0 .. n_chunks, skipping the halves that do not exist; SPG slots per GEMM.
    if (warp == 0 || warp == 2) {
        // ----------------------------------------------------------- weight TMA producers
        // Producer p of each CTA loads the slots with ring position n = p (mod 2): this CTA's
        // half of the rows.  The leader's producer announces the bytes of both halves.
        const uint32_t me = (warp == 0) ? 0u : 1u;
        if (elect_one()) {
            ptx::prefetch_tensormap(&tm_w1);
            ptx::prefetch_tensormap(&tm_w2_128);
            ptx::prefetch_tensormap(&tm_w2_64);
        }
        __syncwarp();
        uint32_t wf_leader;   // w_full[0] of the leader, as a cluster address
        asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(wf_leader) : "r"(MISC_BAR(mb, w_full)));
        auto slot = [&](uint32_t n, const CUtensorMap* tm, int nkb, int rows, int x0, int y) -> bool {
            const uint32_t sl = n % kStages, use = n / kStages;
            const uint32_t we = MISC_BAR(mb, w_empty) + 8u * sl;
            if (!__all_sync(0xffffffffu, ptx::mbar_try_wait(we, (use & 1u) ^ 1u)) &&
                !__all_sync(0xffffffffu, ptx::mbar_wait_slow(we, (use & 1u) ^ 1u, abort_flag)))
                return false;
            if (elect_one()) {
                const uint32_t blk = (uint32_t)rows * 128u;
                const uint32_t dst = wsm + sl * kSlotBytes;
                if (rank == 0) ptx::mbar_arrive_expect_tx(MISC_BAR(mb, w_full) + 8u * sl, 2u * (uint32_t)nkb * blk);
                const uint32_t bar = wf_leader + 8u * sl;
#pragma unroll
                for (int j = 0; j < kMaxKb; ++j)
                    if (j < nkb) ptx::tma_load_2d_pair(dst + (uint32_t)j * blk, tm, x0 + 64 * j, y, bar);
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
                    ffn_tile_lookup(plan, n_lists, pair + (int)ti * n_pairs, kPairRows, l_cur, row0, n_rows);
                }
            }
            if (q < n_chunks) {
                const int y = l_cur * kc_pad + c * C::CH + (int)rank * SS::g1_rows();
#pragma unroll
                for (int i = 0; i < SPG; ++i)
                    if (ok && ((n + i) & 1u) == me)
                        ok = slot(n + i, &tm_w1, SS::g1_nkb(), SS::g1_rows(), 64 * SS::g1_nkb() * i, y);
                n += SPG;
            }
            if (q > 0) {
                const int pl = c ? l_cur : l_last, x = (c ? c - 1 : NC - 1) * C::CH;
#pragma unroll
                for (int i = 0; i < SPG; ++i) {
                    if (!ok || ((n + i) & 1u) != me) continue;
                    if constexpr (D == 128) {
                        ok = slot(n + i, &tm_w2_64, 4, 64, x, pl * D + (int)rank * 64);
                    } else if constexpr (D == 256) {
                        ok = slot(n + i, &tm_w2_128, 2, 128, x + 128 * i, pl * D + (int)rank * 128);
                    } else {
                        if (i == 0) ok = slot(n + i, &tm_w2_128, 2, 128, x, pl * D + (int)rank * 128);
                        else ok = slot(n + i, &tm_w2_64, 2, 64, x, pl * D + 256 + (int)rank * 64);
                    }
                }
                n += SPG;
            }
            if (++c == NC) { c = 0; ++ti; }
        }
    } else if (warp == 1 && rank == 0) {
        // ------------------------------------------------------------------- UMMA issuer
        // As in the single-CTA kernel: one warp of the leader walks the schedule, waits for every
        // slot's barriers, and one elected lane issues every UMMA (one issuing thread: a fixed
        // summation order); every UMMA runs on both CTAs, every commit goes to both.
        constexpr uint32_t idesc256 = ptx::umma_idesc_bf16(256, 256);
        constexpr uint32_t idesc128 = ptx::umma_idesc_bf16(256, 128);
        constexpr uint32_t kBlkLo = kBlockBytes >> 4, kSlotLo = kSlotBytes >> 4;
        const uint32_t tm_h = tmem + C::H_COL0;
        const uint32_t xs_lo = desc_lo(xs), hs_lo = desc_lo(hs), w_lo = desc_lo(wsm);
        auto run = [&](uint32_t n, const SlotWork& w) -> bool {
            const uint32_t sl = n % kStages, ph = (n / kStages) & 1u;
            {
                const uint32_t wf = MISC_BAR(mb, w_full) + 8u * sl;
                bool p = ptx::mbar_try_wait_cluster(wf, ph);
#pragma unroll
                for (int j = 0; j <= kMaxKb; ++j)
                    if (w.wb[j] != 0u) p &= ptx::mbar_try_wait_cluster(w.wb[j], w.wp[j]);
                if (!__all_sync(0xffffffffu, p)) {
                    bool ok = wait_cluster_slow(wf, ph, abort_flag);
#pragma unroll
                    for (int j = 0; j <= kMaxKb; ++j)
                        if (ok && w.wb[j] != 0u) ok = wait_cluster_slow(w.wb[j], w.wp[j], abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) return false;
                }
            }
            ptx::tc_fence_after_sync();   // orders the UMMAs after the other warps' TMEM reads and operand writes
            if (elect_one()) {
                const uint32_t b_lo = w_lo + sl * kSlotLo;
#pragma unroll
                for (int j = 0; j < kMaxKb; ++j)
                    if (j < w.nkb)
                        mma_kblock_pair(w.d_tm, w.a_lo[j], b_lo + (uint32_t)j * w.b_blk_lo, w.idesc,
                                        (j == 0 && w.overwrite) ? 0u : 1u);
#pragma unroll
                for (int j = 0; j <= kMaxKb; ++j)
                    if (w.cb[j] != 0u) ptx::umma_commit_pair(w.cb[j], (uint16_t)3);
                ptx::umma_commit_pair(MISC_BAR(mb, w_empty) + 8u * sl, (uint16_t)3);
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
                    SlotWork w = {};
                    w.d_tm = tm_h;
                    w.idesc = (C::CH == 256) ? idesc256 : idesc128;
                    w.b_blk_lo = (uint32_t)(SS::g1_rows() * 128) >> 4;
                    w.nkb = SS::g1_nkb();
                    w.overwrite = (i == 0);
#pragma unroll
                    for (int j = 0; j < SS::g1_nkb(); ++j) {
                        const uint32_t kb = (uint32_t)(SS::g1_nkb() * i + j);
                        const uint32_t gx = ti * C::KB1 + kb, xslot = gx % C::NXS;
                        w.a_lo[j] = xs_lo + xslot * kBlkLo;
                        if (first) { w.wb[j] = MISC_BAR(mb, x_full) + 8u * xslot; w.wp[j] = (gx / C::NXS) & 1u; }
                        if (last) w.cb[j] = MISC_BAR(mb, x_empty) + 8u * xslot;
                    }
                    if (i == 0) { w.wb[kMaxKb] = MISC_BAR(mb, h_tmem_empty); w.wp[kMaxKb] = hp; }
                    if (i == SPG - 1) w.cb[kMaxKb] = MISC_BAR(mb, h_full);
                    ok = run(n + i, w);
                }
                n += SPG;
            }
            if (q > 0 && ok) {
                // GEMM2 of chunk q-1 = chunk pc of local tile pti:  Y (+)= gelu(H) . W2c_chunk
                const int pc = c ? c - 1 : NC - 1;
                const uint32_t pti = c ? ti : ti - 1, gp = (q - 1) & 1u;
                const bool first = (pc == 0), last = (pc == NC - 1);
                const uint32_t yp = (pti & 1u) ^ 1u;
#pragma unroll
                for (int i = 0; i < SPG; ++i) {
                    if (!ok) continue;
                    SlotWork w = {};
                    w.nkb = SS::g2_nkb();
                    w.b_blk_lo = (uint32_t)(SS::g2_rows(i) * 128) >> 4;
                    if constexpr (D == 128) {
                        w.d_tm = tmem; w.idesc = idesc128; w.overwrite = first;
                    } else if constexpr (D == 256) {
                        w.d_tm = tmem; w.idesc = idesc256; w.overwrite = first && i == 0;
                    } else {
                        w.d_tm = tmem + (i == 0 ? 0u : 256u); w.idesc = (i == 0) ? idesc256 : idesc128; w.overwrite = first;
                    }
#pragma unroll
                    for (int j = 0; j < SS::g2_nkb(); ++j) {
                        const uint32_t hb = (D == 256) ? (uint32_t)(2 * i + j) : (uint32_t)j;   // hidden block
                        w.a_lo[j] = hs_lo + hb * kBlkLo;
                        w.wb[j] = MISC_BAR(mb, hs_full) + 8u * hb; w.wp[j] = gp;
                        // a hidden block is free once the LAST slot that reads it is done
                        if (D != 384 || i == SPG - 1) w.cb[j] = MISC_BAR(mb, hs_empty) + 8u * hb;
                    }
                    // Y's release by the epilogue is needed before the first write of each column range
                    if (first && (i == 0 || D == 384)) { w.wb[kMaxKb] = MISC_BAR(mb, y_empty); w.wp[kMaxKb] = yp; }
                    if (last && i == SPG - 1) w.cb[kMaxKb] = MISC_BAR(mb, y_full);
                    ok = run(n + i, w);
                }
                n += SPG;
            }
            if (++c == NC) { c = 0; ++ti; }
        }
    } else if (warp >= kLoaderWarp0 && warp < kEpiWarp0) {
        // ------------------------------------------------------------------ X row gather
        // This CTA's 128 rows of the tile; a block is published to the leader's barrier once the
        // copies of all lanes have landed.
        const int tl = threadIdx.x - kLoaderWarp0 * 32;
        uint32_t gx = 0, published = 0;
        bool ok = true;
        auto publish_oldest = [&]() {
            cp_async_wait_pending((int)(gx - published) - 1);
            ptx::fence_proxy_async_smem();
            warp_arrive_leader(&misc->x_full[published % C::NXS]);
            ++published;
        };
        for (int t = 0; t < my_tiles && ok; ++t) {
            int l, row0, n_rows;
            ffn_tile_lookup(plan, n_lists, pair + t * n_pairs, kPairRows, l, row0, n_rows);
            row0 += (int)rank * kTileRows;
            n_rows = max(0, min(kTileRows, n_rows - (int)rank * kTileRows));
            int32_t rows[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int r = (tl + j * kLoaderThreads) >> 3;
                rows[j] = r < n_rows ? plan.rowidx[row0 + r] : -1;
            }
            for (int kb = 0; kb < C::KB1 && ok; ++kb) {
                const uint32_t xslot = gx % C::NXS, use = gx / C::NXS;
                uint64_t* bar = &misc->x_empty[xslot];
                while (gx > published &&
                       !__all_sync(0xffffffffu, ptx::mbar_test_wait(ptx::smem_u32(bar), (use & 1u) ^ 1u)))
                    publish_oldest();
                if (!warp_wait(bar, (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int idx = tl + j * kLoaderThreads;
                    const int r = idx >> 3, ci = idx & 7;
                    const uint32_t dst = xs + xslot * kBlockBytes + r * 128 + ((ci ^ (r & 7)) << 4);
                    if (rows[j] >= 0) {
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
        uint32_t g = 0;
        bool ok = true;
        int32_t my_row = -1, prev_row = -1;
        constexpr int kDrainBlk = C::NBATCH - 1;
        const uint32_t stg = hs + (uint32_t)(half * C::NBATCH + kDrainBlk) * kBlockBytes + (uint32_t)quarter * 4096u;
        auto drain_y = [&](uint32_t t_idx, int32_t grow) {
            if (!warp_wait(&misc->y_full, t_idx & 1u, abort_flag)) { ok = false; return; }
            ptx::tc_fence_after_sync();
            // 64 columns per pass: two TMEM loads and one wait, bf16 rows through the staging
            // piece, then whole 128-byte row segments to global memory.  The registers a TMEM
            // load writes are not named again before its wait.
            constexpr int NP = D / 128;
            const int ch = lane & 7;
            int32_t grs[8];
#pragma unroll
            for (int step = 0; step < 8; ++step) grs[step] = __shfl_sync(0xffffffffu, grow, step * 4 + (lane >> 3));
            __nv_bfloat16* ycol = Y + half * (D / 2) + ch * 8;
#pragma unroll 1
            for (int pass = 0; pass < NP; ++pass) {
                uint32_t ra[32], rb[32];
                const int col0 = half * (D / 2) + pass * 64;
                ptx::tmem_ld_32x32(lane_base + col0, ra);
                ptx::tmem_ld_32x32(lane_base + col0 + 32, rb);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + ((i ^ (lane & 7)) << 4)),
                                 "r"(pack_bf16x2(__uint_as_float(ra[8 * i]), __uint_as_float(ra[8 * i + 1]))),
                                 "r"(pack_bf16x2(__uint_as_float(ra[8 * i + 2]), __uint_as_float(ra[8 * i + 3]))),
                                 "r"(pack_bf16x2(__uint_as_float(ra[8 * i + 4]), __uint_as_float(ra[8 * i + 5]))),
                                 "r"(pack_bf16x2(__uint_as_float(ra[8 * i + 6]), __uint_as_float(ra[8 * i + 7])))
                                 : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((4 + i) ^ (lane & 7)) << 4)),
                                 "r"(pack_bf16x2(__uint_as_float(rb[8 * i]), __uint_as_float(rb[8 * i + 1]))),
                                 "r"(pack_bf16x2(__uint_as_float(rb[8 * i + 2]), __uint_as_float(rb[8 * i + 3]))),
                                 "r"(pack_bf16x2(__uint_as_float(rb[8 * i + 4]), __uint_as_float(rb[8 * i + 5]))),
                                 "r"(pack_bf16x2(__uint_as_float(rb[8 * i + 6]), __uint_as_float(rb[8 * i + 7])))
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
            warp_arrive_leader(&misc->y_empty);
        };
        for (int t = 0; t < my_tiles && ok; ++t) {
            int l, row0, n_rows;
            ffn_tile_lookup(plan, n_lists, pair + t * n_pairs, kPairRows, l, row0, n_rows);
            row0 += (int)rank * kTileRows;
            n_rows = max(0, min(kTileRows, n_rows - (int)rank * kTileRows));
            prev_row = my_row;
            my_row = row < n_rows ? plan.rowidx[row0 + row] : -1;
            for (int c = 0; c < NC && ok; ++c, ++g) {
                if (!warp_wait(&misc->h_full, g & 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int j = 0; j < C::NBATCH && ok; ++j) {
                    const int blk = half * C::NBATCH + j;
                    // Y of the previous tile is complete about now (its last GEMM2 was queued right
                    // after this tile's first GEMM1): store it before this warp's last batch of the
                    // chunk is loaded, while no accumulator values are held in registers
                    if (j == C::NBATCH - 1 && c == 0 && t > 0) {
                        drain_y((uint32_t)(t - 1), prev_row);
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
                        warp_arrive_leader(&misc->h_tmem_empty);
                    }
                    uint32_t pk[32];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        pk[i] = gelu_erf_fast_bf16x2(__uint_as_float(h0[2 * i]), __uint_as_float(h0[2 * i + 1]));
                        pk[16 + i] = gelu_erf_fast_bf16x2(__uint_as_float(h1[2 * i]), __uint_as_float(h1[2 * i + 1]));
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
                    warp_arrive_leader(&misc->hs_full[blk]);
                }
            }
        }
        if (ok && my_tiles > 0) drain_y((uint32_t)(my_tiles - 1), my_row);
    }

    // ---------------------------------------------------------------------------- teardown
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_TIMEOUT);
        // give copies and UMMAs still in flight time to land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
        __syncthreads();
    }
    // neither CTA may leave while the other can still signal its barriers or read its operands
    ptx::cluster_sync_all();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem, kTmemCols);
    }
}

template <int D>
int launch_d(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c, int kc_pad,
             int max_tiles, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    CUtensorMap m1, m2a, m2b;
    const uint64_t r1 = (uint64_t)d.n_lists * kc_pad, r2 = (uint64_t)d.n_lists * D;
    if (!make_weight_map(&m1, w1c, r1, D, SlotShape<D>::g1_rows())) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2a, w2c, r2, kc_pad, 128)) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2b, w2c, r2, kc_pad, 64)) return SENTRY_ERR_CUDA;
    auto kern = ffn_tc_pair_kernel<D>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::SMEM_BYTES));
    int pairs = ctx->sm_count / 2;
    if (max_tiles < pairs) pairs = max_tiles;
    if (pairs < 1) pairs = 1;
    LaunchScope ls(ctx, KS_FFN_MAIN, st);
    kern<<<2 * pairs, kThreads, Cfg<D>::SMEM_BYTES, st>>>(m1, m2a, m2b, (const __nv_bfloat16*)a.X,
                                                           (__nv_bfloat16*)a.Y, plan, d.n_lists, kc_pad, a.status);
    return SENTRY_OK;
}

}  // namespace

int ffn_tc_pair_tile_rows() { return kPairRows; }

// `max_tiles`: upper bound on the number of 256-row tiles of the plan.
int launch_ffn_tc_pair(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c,
                       int kc_pad, int max_tiles, cudaStream_t st) {
    int rc;
    switch (a.d.D) {
        case 128: rc = launch_d<128>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st); break;
        case 256: rc = launch_d<256>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st); break;
        case 384: rc = launch_d<384>(ctx, a, plan, w1c, w2c, kc_pad, max_tiles, st); break;
        default: return SENTRY_ERR_UNSUPPORTED;
    }
    if (rc != SENTRY_OK) return rc;
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

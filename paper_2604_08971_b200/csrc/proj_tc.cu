// Projections of the pruned layer (Section 4.6, head pruning with GQA consistency) for bf16 on
// the 5th-generation tensor cores.  One CTA per (sample, tile of 128 present tokens).
//
//   QKV   A = the tile's X rows, gathered once into shared memory (K-major, 128-byte swizzle).
//         Every kept head, and K and V of every referenced KV group, is one "slice": its column
//         block W[:, i d:(i+1) d] streams through a ring of TMA stages as it lies in memory (rows =
//         d_model index, i.e. an MN-major B operand) and is multiplied into its own d columns of
//         tensor memory.  Pruned heads and unreferenced groups are never fetched.
//   OUT   A = the tile's rows of every kept head's attention output (d wide each); the slice of
//         head h is the row block W_O[h d:(h+1) d, :], accumulated into one [128 x d_model] tile.
// Warp 0 feeds the weight ring, warp 1 issues the UMMAs, warps 4-7 read the accumulators and store.
// Every wait is bounded; on expiry the CTA raises SENTRY_STATUS_BIT_TIMEOUT and unwinds.
#include <cuda.h>

#include "attend_common.cuh"
#include "tc_common.cuh"

// Compiled a second time for IEEE-half tensors (proj_tc_f16.cu): the operand format of the UMMAs
// and the packing of the results (pack2, attend_common.cuh) are what differs.
#ifdef SENTRY_ATT_F16
#define PROJ_IDESC ptx::umma_idesc_f16_major
#else
#define PROJ_IDESC ptx::umma_idesc_bf16_major
#endif

namespace {

constexpr int kPThreads = 256;
constexpr int kPStages = 3;
constexpr int kMaxSlicesTc = 96;

struct ProjMisc {
    uint64_t w_full[kPStages], w_empty[kPStages];
    uint64_t acc_full, acc_empty;
    uint32_t tmem_base;
    int abort_flag;
    int n_slices;
    int kind[kMaxSlicesTc], idx[kMaxSlicesTc];   // QKV: 0 = Q head, 1 = K group, 2 = V group.  OUT: kept-list slot, head
};

// ------------------------------------------------------------------------------------- QKV
// dynamic smem: X tile [D/64][128 x 128 B] | weight ring [kPStages][D x DH] | misc | valid list
template <int DH>
__global__ void __launch_bounds__(kPThreads, 1)
proj_qkv_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __nv_bfloat16* __restrict__ X,
                   const int32_t* __restrict__ kept_heads, const int32_t* __restrict__ ids,
                   const uint32_t* __restrict__ masks, int Tlen, int D, int Hq, int Hk, int k_h,
                   __nv_bfloat16* __restrict__ Q, __nv_bfloat16* __restrict__ K, __nv_bfloat16* __restrict__ V,
                   unsigned int* status) {
    constexpr int RB = DH * 2;
    constexpr int NS = 512 / DH;                    // slices whose accumulators fit in tensor memory at once
    extern __shared__ uint8_t smem_raw[];
    __shared__ int red[66];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    const int KB = D / 64;
    const uint32_t stage_bytes = (uint32_t)D * RB;
    const uint32_t xs = base, wsm = base + (uint32_t)KB * 16384u;
    ProjMisc* misc = reinterpret_cast<ProjMisc*>(smem + (size_t)KB * 16384 + (size_t)kPStages * stage_bytes);
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(misc) + ((sizeof(ProjMisc) + 127) / 128) * 128);
    volatile int* abort_flag = &misc->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_per_sample = (Tlen + 127) / 128;
    const int b = blockIdx.x / tiles_per_sample, tt = blockIdx.x % tiles_per_sample;

    const int Tv = block_build_valid(ids, Tlen, masks[b], s_valid, red);
    if (tt * 128 >= Tv) return;                      // no present token in this tile
    const int n_rows = min(128, Tv - tt * 128);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->w_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->acc_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->acc_empty), 4);
        misc->abort_flag = 0;
        ptx::fence_barrier_init();
        const int r = Hq / Hk;
        int n = 0;
        uint32_t groups = 0;
        for (int j = 0; j < k_h; ++j) {
            const int h = kept_heads[(size_t)b * k_h + j];
            if (h < 0 || h >= Hq) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); continue; }
            misc->kind[n] = 0; misc->idx[n] = h; ++n;
            groups |= 1u << (h / r);
        }
        for (int g = 0; g < Hk; ++g)
            if ((groups >> g) & 1u) {
                misc->kind[n] = 1; misc->idx[n] = g; ++n;
                misc->kind[n] = 2; misc->idx[n] = g; ++n;
            }
        misc->n_slices = n;
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), 512);
        ptx::tmem_relinquish();
    }
    // the tile's X rows: 16-byte chunk ci of row r of block kb at  r * 128 + ((ci ^ (r & 7)) << 4)
    for (int i = threadIdx.x; i < KB * 128 * 8; i += blockDim.x) {
        const int kb = i / 1024, r = (i >> 3) & 127, ci = i & 7;
        const uint32_t dst = xs + (uint32_t)kb * 16384u + (uint32_t)r * 128u + (uint32_t)((ci ^ (r & 7)) << 4);
        if (r < n_rows) {
            const int tok = s_valid[tt * 128 + r];
            ptx::cp_async_16(dst, X + ((size_t)b * Tlen + tok) * D + kb * 64 + ci * 8);
        } else {
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
        }
    }
    ptx::cp_async_wait_all();
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = misc->tmem_base;
    const int n_slices = misc->n_slices;

    if (warp == 0) {
        // ------------------------------------------------------------ weight producer
        bool ok = true;
        for (int s = 0; s < n_slices && ok; ++s) {
            const uint32_t st = (uint32_t)s % kPStages, use = (uint32_t)s / kPStages;
            ok = warp_wait(&misc->w_empty[st], (use & 1u) ^ 1u, abort_flag);
            if (!ok) break;
            if (elect_one()) {
                const int kind = misc->kind[s], idx = misc->idx[s];
                const CUtensorMap* tm = kind == 0 ? &tm_q : (kind == 1 ? &tm_k : &tm_v);
                const uint32_t bar = ptx::smem_u32(&misc->w_full[st]);
                ptx::mbar_arrive_expect_tx(bar, stage_bytes);
                for (int kb = 0; kb < KB; ++kb)
                    ptx::tma_load_2d(wsm + st * stage_bytes + (uint32_t)kb * 64u * RB, tm, idx * DH, kb * 64, bar);
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc = PROJ_IDESC(128, DH, false, true);
        bool ok = true;
        for (int s = 0; s < n_slices && ok; ++s) {
            const uint32_t st = (uint32_t)s % kPStages, use = (uint32_t)s / kPStages;
            const int grp = s / NS;
            if (s % NS == 0 && grp > 0) ok = warp_wait(&misc->acc_empty, ((uint32_t)(grp - 1)) & 1u, abort_flag);
            if (ok) ok = warp_wait(&misc->w_full[st], use & 1u, abort_flag);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (elect_one()) {
                const uint32_t d_tm = tmem + (uint32_t)(s % NS) * DH;
                for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t a = ptx::umma_smem_desc_sw128(xs + (uint32_t)kb * 16384u + ks * 32);
                        const uint64_t bd = ptx::umma_smem_desc_rows(
                            wsm + st * stage_bytes + (uint32_t)(kb * 64 + ks * 16) * RB, RB);
                        ptx::umma_bf16(d_tm, a, bd, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                    }
                }
                ptx::umma_commit(ptx::smem_u32(&misc->w_empty[st]));
                if (s % NS == NS - 1 || s == n_slices - 1) ptx::umma_commit(ptx::smem_u32(&misc->acc_full));
            }
            __syncwarp();
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------- epilogue
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const int tok = row < n_rows ? (int)s_valid[tt * 128 + row] : -1;
        const int n_groups = (n_slices + NS - 1) / NS;
        bool ok = true;
        for (int grp = 0; grp < n_groups && ok; ++grp) {
            ok = warp_wait(&misc->acc_full, (uint32_t)grp & 1u, abort_flag);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const int s_end = min(n_slices, (grp + 1) * NS);
            for (int s = grp * NS; s < s_end; ++s) {
                uint32_t acc[DH];
                if constexpr (DH == 16) {
                    ptx::tmem_ld_32x16(lane_base + (uint32_t)(s % NS) * DH, reinterpret_cast<uint32_t(&)[16]>(acc));
                } else {
#pragma unroll
                    for (int j = 0; j < DH / 32; ++j)
                        ptx::tmem_ld_32x32(lane_base + (uint32_t)(s % NS) * DH + 32 * j,
                                           reinterpret_cast<uint32_t(&)[32]>(acc[32 * j]));
                }
                ptx::tmem_ld_wait();
                if (tok >= 0) {
                    const int kind = misc->kind[s], idx = misc->idx[s];
                    __nv_bfloat16* dst = kind == 0 ? Q + (((size_t)b * Hq + idx) * Tlen + tok) * DH
                                                   : (kind == 1 ? K : V) + (((size_t)b * Hk + idx) * Tlen + tok) * DH;
#pragma unroll
                    for (int cc = 0; cc < DH / 8; ++cc) {
                        uint4 v;
                        v.x = pack2(__uint_as_float(acc[8 * cc]), __uint_as_float(acc[8 * cc + 1]));
                        v.y = pack2(__uint_as_float(acc[8 * cc + 2]), __uint_as_float(acc[8 * cc + 3]));
                        v.z = pack2(__uint_as_float(acc[8 * cc + 4]), __uint_as_float(acc[8 * cc + 5]));
                        v.w = pack2(__uint_as_float(acc[8 * cc + 6]), __uint_as_float(acc[8 * cc + 7]));
                        reinterpret_cast<uint4*>(dst)[cc] = v;
                    }
                }
            }
            ptx::tc_fence_before_sync();
            warp_arrive(&misc->acc_empty);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_TIMEOUT);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512);
    }
}

// ------------------------------------------------------------------------------------- OUT
// dynamic smem: A tiles [k_h][128 x DH] | weight ring [kPStages][DH x D] | misc | valid list
template <int DH>
__global__ void __launch_bounds__(kPThreads, 1)
proj_out_tc_kernel(const __grid_constant__ CUtensorMap tm_o, const __nv_bfloat16* __restrict__ A,
                   const int32_t* __restrict__ kept_heads, const int32_t* __restrict__ ids,
                   const uint32_t* __restrict__ masks, int Tlen, int D, int Hq, int k_h,
                   __nv_bfloat16* __restrict__ out, unsigned int* status) {
    using S = Sw<DH>;
    constexpr int RB = DH * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ int red[66];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    const int NC = D / 64;
    const uint32_t stage_bytes = (uint32_t)D * RB;
    const uint32_t a_tile = 128u * RB;
    const uint32_t as = base, wsm = base + (uint32_t)k_h * a_tile;
    ProjMisc* misc = reinterpret_cast<ProjMisc*>(smem + (size_t)k_h * a_tile + (size_t)kPStages * stage_bytes);
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(misc) + ((sizeof(ProjMisc) + 127) / 128) * 128);
    volatile int* abort_flag = &misc->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_per_sample = (Tlen + 127) / 128;
    const int b = blockIdx.x / tiles_per_sample, tt = blockIdx.x % tiles_per_sample;
    const uint32_t mask = masks[b];

    // rows of absent tokens are zero: every CTA clears those among its 128 token positions
    {
        const int vpr = D / 8;
        for (int i = threadIdx.x; i < 128 * vpr; i += blockDim.x) {
            const int t = tt * 128 + i / vpr;
            if (t >= Tlen) break;
            const int m = ids[t];
            if (!(m >= 0 && m < 32 && ((mask >> m) & 1u)))
                reinterpret_cast<uint4*>(out + ((size_t)b * Tlen + t) * D)[i % vpr] = make_uint4(0, 0, 0, 0);
        }
    }
    const int Tv = block_build_valid(ids, Tlen, mask, s_valid, red);
    if (tt * 128 >= Tv) return;
    const int n_rows = min(128, Tv - tt * 128);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->w_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->acc_full), 1);
        misc->abort_flag = 0;
        ptx::fence_barrier_init();
        int n = 0;
        for (int j = 0; j < k_h; ++j) {
            const int h = kept_heads[(size_t)b * k_h + j];
            if (h < 0 || h >= Hq) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); continue; }
            misc->kind[n] = j; misc->idx[n] = h; ++n;
        }
        misc->n_slices = n;
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), 512);
        ptx::tmem_relinquish();
    }
    // the tile's rows of every kept head's attention output
    for (int i = threadIdx.x; i < k_h * 128 * S::CPR; i += blockDim.x) {
        const int j = i / (128 * S::CPR), r = (i / S::CPR) % 128, cc = i % S::CPR;
        const uint32_t dst = as + (uint32_t)j * a_tile + S::off(r, cc);
        if (r < n_rows) {
            const int tok = s_valid[tt * 128 + r];
            ptx::cp_async_16(dst, A + (((size_t)b * k_h + j) * Tlen + tok) * DH + cc * 8);
        } else {
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
        }
    }
    ptx::cp_async_wait_all();
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = misc->tmem_base;
    const int n_slices = misc->n_slices;

    if (warp == 0) {
        bool ok = true;
        for (int s = 0; s < n_slices && ok; ++s) {
            const uint32_t st = (uint32_t)s % kPStages, use = (uint32_t)s / kPStages;
            ok = warp_wait(&misc->w_empty[st], (use & 1u) ^ 1u, abort_flag);
            if (!ok) break;
            if (elect_one()) {
                const uint32_t bar = ptx::smem_u32(&misc->w_full[st]);
                ptx::mbar_arrive_expect_tx(bar, stage_bytes);
                for (int nc = 0; nc < NC; ++nc)   // 64 output columns x DH rows of W_O per box
                    ptx::tma_load_2d(wsm + st * stage_bytes + (uint32_t)nc * DH * 128u, &tm_o, nc * 64, misc->idx[s] * DH, bar);
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        constexpr uint32_t idesc = PROJ_IDESC(128, 64, false, true);
        bool ok = true;
        for (int s = 0; s < n_slices && ok; ++s) {
            const uint32_t st = (uint32_t)s % kPStages, use = (uint32_t)s / kPStages;
            ok = warp_wait(&misc->w_full[st], use & 1u, abort_flag);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (elect_one()) {
                const uint32_t a0 = as + (uint32_t)misc->kind[s] * a_tile;
                for (int nc = 0; nc < NC; ++nc) {
#pragma unroll
                    for (int ks = 0; ks < DH / 16; ++ks) {
                        const uint64_t a = ptx::umma_smem_desc_rows(a0 + ks * 32, RB);
                        const uint64_t bd = ptx::umma_smem_desc_rows(
                            wsm + st * stage_bytes + (uint32_t)nc * DH * 128u + (uint32_t)ks * 16u * 128u, 128);
                        ptx::umma_bf16(tmem + (uint32_t)nc * 64, a, bd, idesc, (s > 0 || ks > 0) ? 1u : 0u);
                    }
                }
                ptx::umma_commit(ptx::smem_u32(&misc->w_empty[st]));
                if (s == n_slices - 1) ptx::umma_commit(ptx::smem_u32(&misc->acc_full));
            }
            __syncwarp();
        }
    } else if (warp >= 4) {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const int tok = row < n_rows ? (int)s_valid[tt * 128 + row] : -1;
        if (n_slices > 0 && warp_wait(&misc->acc_full, 0u, abort_flag)) {
            ptx::tc_fence_after_sync();
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t acc[32];
                ptx::tmem_ld_32x32(lane_base + c0, acc);
                ptx::tmem_ld_wait();
                if (tok >= 0) {
                    uint4* dst = reinterpret_cast<uint4*>(out + ((size_t)b * Tlen + tok) * D + c0);
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint4 v;
                        v.x = pack2(__uint_as_float(acc[8 * cc]), __uint_as_float(acc[8 * cc + 1]));
                        v.y = pack2(__uint_as_float(acc[8 * cc + 2]), __uint_as_float(acc[8 * cc + 3]));
                        v.z = pack2(__uint_as_float(acc[8 * cc + 4]), __uint_as_float(acc[8 * cc + 5]));
                        v.w = pack2(__uint_as_float(acc[8 * cc + 6]), __uint_as_float(acc[8 * cc + 7]));
                        dst[cc] = v;
                    }
                }
            }
        } else if (n_slices == 0 && tok >= 0) {   // no valid kept head: the rows are zero
            for (int c0 = 0; c0 < D; c0 += 8)
                *reinterpret_cast<uint4*>(out + ((size_t)b * Tlen + tok) * D + c0) = make_uint4(0, 0, 0, 0);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_TIMEOUT);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, 512);
    }
}

size_t out_smem_bytes(int D, int DH, int k_h, int T) {
    return (size_t)k_h * 128 * DH * 2 + (size_t)kPStages * D * DH * 2 + ((sizeof(ProjMisc) + 127) / 128) * 128 +
           ((size_t)T * 2 + 127) / 128 * 128 + 1024;
}

template <int DH>
int launch_out_d(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st) {
    const sentry_proj_desc& d = a.d;
    CUtensorMap mo;
    if (!make_map_2d(&mo, a.WO, (uint64_t)d.Hq * DH, d.D, DH, 64)) return SENTRY_ERR_CUDA;
    const size_t smem = out_smem_bytes(d.D, DH, d.k_h, d.T);
    auto kern = proj_out_tc_kernel<DH>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned grid = (unsigned)((size_t)d.B * ((d.T + 127) / 128));
    LaunchScope ls(ctx, KS_PROJ_OUT, st);
    kern<<<grid, kPThreads, smem, st>>>(mo, (const __nv_bfloat16*)a.A, a.kept_heads, a.ids, a.masks, d.T, d.D, d.Hq,
                                        d.k_h, (__nv_bfloat16*)a.out, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

size_t qkv_smem_bytes(int D, int DH, int T) {
    return (size_t)(D / 64) * 16384 + (size_t)kPStages * D * DH * 2 + ((sizeof(ProjMisc) + 127) / 128) * 128 +
           ((size_t)T * 2 + 127) / 128 * 128 + 1024;
}

template <int DH>
int launch_qkv_d(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st) {
    const sentry_proj_desc& d = a.d;
    CUtensorMap mq, mk, mv;
    if (!make_map_2d(&mq, a.WQ, d.D, (uint64_t)d.Hq * DH, 64, DH) || !make_map_2d(&mk, a.WK, d.D, (uint64_t)d.Hk * DH, 64, DH) ||
        !make_map_2d(&mv, a.WV, d.D, (uint64_t)d.Hk * DH, 64, DH))
        return SENTRY_ERR_CUDA;
    const size_t smem = qkv_smem_bytes(d.D, DH, d.T);
    auto kern = proj_qkv_tc_kernel<DH>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned grid = (unsigned)((size_t)d.B * ((d.T + 127) / 128));
    LaunchScope ls(ctx, KS_PROJ_QKV, st);
    kern<<<grid, kPThreads, smem, st>>>(mq, mk, mv, (const __nv_bfloat16*)a.X, a.kept_heads, a.ids, a.masks, d.T, d.D,
                                        d.Hq, d.Hk, d.k_h, (__nv_bfloat16*)a.Q, (__nv_bfloat16*)a.K,
                                        (__nv_bfloat16*)a.V, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

}  // namespace

// bf16, head dim 16/32/64, d_model a multiple of 64, everything within one SM's shared memory,
// and one CTA's tile count within the grid limit
bool project_qkv_tc_supported(const sentry_proj_desc& d) {
    if (d.dtype != ATT_DTYPE) return false;
    if (d.d != 16 && d.d != 32 && d.d != 64) return false;
    if (d.D % 64 != 0 || d.T > 65535) return false;
    if (d.k_h + 2 * d.Hk > kMaxSlicesTc) return false;
    return qkv_smem_bytes(d.D, d.d, d.T) <= 220 * 1024;
}

int launch_project_qkv_tc(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st) {
    switch (a.d.d) {
        case 16: return launch_qkv_d<16>(ctx, a, st);
        case 32: return launch_qkv_d<32>(ctx, a, st);
        case 64: return launch_qkv_d<64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

bool project_out_tc_supported(const sentry_proj_desc& d) {
    if (d.dtype != ATT_DTYPE) return false;
    if (d.d != 16 && d.d != 32 && d.d != 64) return false;
    if (d.D % 64 != 0 || d.D > 512 || d.T > 65535 || d.k_h > kMaxSlicesTc) return false;
    return out_smem_bytes(d.D, d.d, d.k_h, d.T) <= 220 * 1024;
}

int launch_project_out_tc(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st) {
    switch (a.d.d) {
        case 16: return launch_out_d<16>(ctx, a, st);
        case 32: return launch_out_d<32>(ctx, a, st);
        case 64: return launch_out_d<64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

// Channel-compacted FFN on the 5th-generation tensor cores (Section 4.6):
//   Y = gelu(X . W1[:, N]) . W2[N, :]   for the present rows of every sample.
//
// One persistent CTA per SM walks tiles of 128 present rows (row plan in ffn_plan.cuh).
// Per tile and per chunk of 128 kept channels:
//   GEMM1  H[128 x 128] = X_tile[128 x D] . W1c_chunk^T          (tcgen05, fp32 in TMEM)
//   epilogue  H -> gelu -> bf16 -> shared memory (K-major, 128-byte swizzle)
//   GEMM2  Y[128 x D] += H[128 x 128] . W2c_chunk                 (tcgen05, fp32 in TMEM)
// The hidden activations never leave the SM.  Weights are the gathered, K-major copies made
// by the prepack kernel; 128 x 64 tiles of them stream through a TMA ring.  X rows are
// gathered with 16-byte async copies into the same swizzled layout TMA would produce.
//
// Warp roles (384 threads): warp 0 = weight TMA producer and TMEM owner, warp 1 = UMMA
// issuer, warps 2-3 = X row gather, warps 4-11 = epilogue (two warps per TMEM lane quarter).
// Every wait is bounded; on expiry the CTA raises SENTRY_STATUS_BIT_TIMEOUT and unwinds.
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "ffn_plan.cuh"
#include "ptx/sm100.cuh"

namespace {

constexpr int kTileRows = 128;
constexpr int kChunk = 128;            // kept channels per chunk
constexpr int kStageBytes = 128 * 128; // one 128-row x 64-element bf16 weight tile
constexpr int kHBytes = 128 * 128 * 2; // hidden chunk, bf16
constexpr int kThreads = 384;
constexpr int kEpiThreads = 256;
constexpr int kLoaderThreads = 64;
constexpr int kTmemCols = 512;

template <int D>
struct Cfg {
    static constexpr int KB1 = D / 64;               // K blocks of GEMM1
    static constexpr int NB2 = D / 128;              // N blocks of GEMM2
    static constexpr int NHBUF = (D <= 256) ? 2 : 1; // hidden-chunk buffers (TMEM and smem)
    static constexpr int NSTAGES = (D == 128) ? 6 : 5;
    static constexpr int X_BYTES = kTileRows * D * 2;
    static constexpr int H_COL0 = (D <= 256) ? 256 : 384;  // TMEM column of hidden buffer 0
    static constexpr int OFF_H = X_BYTES;
    static constexpr int OFF_W = OFF_H + NHBUF * kHBytes;
    static constexpr int OFF_MISC = OFF_W + NSTAGES * kStageBytes;
    static constexpr int SMEM_BYTES = OFF_MISC + 2048 + 1024;  // + misc + alignment slack
};

struct Misc {
    uint64_t w_full[8], w_empty[8];
    uint64_t x_full, x_empty;
    uint64_t h_full[2], h_tmem_empty[2], hs_full[2], hs_empty[2];
    uint64_t y_full, y_empty;
    uint32_t tmem_base;
    int abort_flag;
    int32_t row[2][kTileRows];
};
static_assert(sizeof(Misc) <= 2048, "misc block too large");

__device__ __forceinline__ float gelu_erf(float z) {
    return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap tm_w1, const __grid_constant__ CUtensorMap tm_w2,
              const __nv_bfloat16* __restrict__ X, __nv_bfloat16* __restrict__ Y, FfnPlan plan,
              int n_lists, int Tlen, int kc_pad, unsigned int* status) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;   // 1024-byte aligned tile base
    uint8_t* smem = smem_raw + (base - raw_addr);
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);
    const uint32_t xs = base, hs = base + C::OFF_H, wsm = base + C::OFF_W;
    volatile int* abort_flag = &misc->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NC = kc_pad / kChunk;
    const int total_tiles = plan.tile_start[n_lists];

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::NSTAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&misc->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->w_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->x_full), kLoaderThreads);
        ptx::mbar_init(ptx::smem_u32(&misc->x_empty), 1);
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&misc->h_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->h_tmem_empty[b]), kEpiThreads);
            ptx::mbar_init(ptx::smem_u32(&misc->hs_full[b]), kEpiThreads);
            ptx::mbar_init(ptx::smem_u32(&misc->hs_empty[b]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->y_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->y_empty), kEpiThreads);
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

    if (warp == 0) {
        // ------------------------------------------------------------ weight TMA producer
        if (lane == 0) {
            ptx::prefetch_tensormap(&tm_w1);
            ptx::prefetch_tensormap(&tm_w2);
            uint32_t n = 0;
            bool ok = true;
            auto issue = [&](const CUtensorMap* tm, int x, int y) {
                const uint32_t s = n % C::NSTAGES, use = n / C::NSTAGES;
                if (!ptx::mbar_wait(ptx::smem_u32(&misc->w_empty[s]), (use & 1u) ^ 1u, abort_flag)) {
                    ok = false;
                    return;
                }
                const uint32_t bar = ptx::smem_u32(&misc->w_full[s]);
                ptx::mbar_arrive_expect_tx(bar, kStageBytes);
                ptx::tma_load_2d(wsm + s * kStageBytes, tm, x, y, bar);
                ++n;
            };
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                int l, slot0, n_rows;
                ffn_tile_lookup(plan, n_lists, tile, kTileRows, l, slot0, n_rows);
                for (int c = 0; c <= NC && ok; ++c) {
                    if (c < NC)
                        for (int kb = 0; kb < C::KB1 && ok; ++kb)
                            issue(&tm_w1, kb * 64, l * kc_pad + c * kChunk);
                    if (c > 0)
                        for (int nb = 0; nb < C::NB2 && ok; ++nb)
                            for (int kb2 = 0; kb2 < 2 && ok; ++kb2)
                                issue(&tm_w2, (c - 1) * kChunk + kb2 * 64, l * D + nb * 128);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------- UMMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(128, 128);
            uint32_t n = 0, hc = 0, ti = 0;
            bool ok = true;
            auto wait = [&](uint64_t* bar, uint32_t parity) {
                if (ok && !ptx::mbar_wait(ptx::smem_u32(bar), parity, abort_flag)) ok = false;
                ptx::tc_fence_after_sync();
                return ok;
            };
            // one 128x128x64 block: A tile at a_addr, B = current weight stage
            auto block = [&](uint32_t d_tmem, uint32_t a_addr, bool first) {
                const uint32_t s = n % C::NSTAGES, use = n / C::NSTAGES;
                if (!wait(&misc->w_full[s], use & 1u)) return;
                const uint64_t ad = ptx::umma_smem_desc_sw128(a_addr);
                const uint64_t bd = ptx::umma_smem_desc_sw128(wsm + s * kStageBytes);
#pragma unroll
                for (uint32_t ks = 0; ks < 4; ++ks)
                    ptx::umma_bf16(d_tmem, ad + 2u * ks, bd + 2u * ks, idesc, (!first || ks > 0) ? 1u : 0u);
                ptx::umma_commit(ptx::smem_u32(&misc->w_empty[s]));
                ++n;
            };
            auto gemm2 = [&](int cc) {
                const uint32_t g = hc + cc, buf = g % C::NHBUF, use = g / C::NHBUF;
                if (!wait(&misc->hs_full[buf], use & 1u)) return;
                if (cc == 0 && !wait(&misc->y_empty, (ti & 1u) ^ 1u)) return;
                for (int nb = 0; nb < C::NB2 && ok; ++nb)
                    for (int kb2 = 0; kb2 < 2 && ok; ++kb2)
                        block(tmem + nb * 128, hs + buf * kHBytes + kb2 * 16384, cc == 0 && kb2 == 0);
                if (ok) ptx::umma_commit(ptx::smem_u32(&misc->hs_empty[buf]));
            };
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++ti) {
                if (!wait(&misc->x_full, ti & 1u)) break;
                for (int c = 0; c < NC && ok; ++c) {
                    const uint32_t g = hc + c, buf = g % C::NHBUF, use = g / C::NHBUF;
                    if (!wait(&misc->h_tmem_empty[buf], (use & 1u) ^ 1u)) break;
                    for (int kb = 0; kb < C::KB1 && ok; ++kb)
                        block(tmem + C::H_COL0 + buf * 128, xs + kb * 16384, kb == 0);
                    if (!ok) break;
                    ptx::umma_commit(ptx::smem_u32(&misc->h_full[buf]));
                    if (c == NC - 1) ptx::umma_commit(ptx::smem_u32(&misc->x_empty));
                    if (c > 0) gemm2(c - 1);
                }
                if (ok) gemm2(NC - 1);
                if (ok) ptx::umma_commit(ptx::smem_u32(&misc->y_full));
                hc += NC;
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------------ X row gather
        const int t64 = threadIdx.x - 64;
        constexpr int CH = D / 8;  // 16-byte chunks per row
        uint32_t ti = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++ti) {
            int l, slot0, n_rows;
            ffn_tile_lookup(plan, n_lists, tile, kTileRows, l, slot0, n_rows);
            // x_empty also orders this write after the epilogue's read of the buffer two tiles back
            if (!ptx::mbar_wait(ptx::smem_u32(&misc->x_empty), (ti & 1u) ^ 1u, abort_flag)) break;
            int32_t* rowbuf = misc->row[ti & 1u];
            for (int r = t64; r < kTileRows; r += kLoaderThreads)
                rowbuf[r] = r < n_rows ? (int32_t)ffn_row_of_slot(plan, l, slot0 + r, Tlen) : -1;
            asm volatile("bar.sync 1, 64;" ::: "memory");
            for (int idx = t64; idx < kTileRows * CH; idx += kLoaderThreads) {
                const int r = idx / CH, ci = idx % CH;
                const uint32_t dst = xs + (ci >> 3) * 16384 + r * 128 + (((ci & 7) ^ (r & 7)) << 4);
                const int32_t grow = rowbuf[r];
                if (grow >= 0) {
                    ptx::cp_async_16(dst, X + (size_t)grow * D + ci * 8);
                } else {
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
                }
            }
            ptx::cp_async_wait_all();
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(ptx::smem_u32(&misc->x_full));
        }
    } else {
        // ---------------------------------------------------------------------- epilogue
        const int quarter = warp & 3, half = (warp - 4) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        uint32_t hc = 0, ti = 0;
        bool ok = true;
        uint32_t r[32];
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++ti) {
            int32_t my_row = -1;
            for (int c = 0; c < NC; ++c) {
                const uint32_t g = hc + c, buf = g % C::NHBUF, use = g / C::NHBUF;
                if (!ptx::mbar_wait(ptx::smem_u32(&misc->h_full[buf]), use & 1u, abort_flag)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                if (c == 0) my_row = misc->row[ti & 1u][row];
                if (!ptx::mbar_wait(ptx::smem_u32(&misc->hs_empty[buf]), (use & 1u) ^ 1u, abort_flag)) { ok = false; break; }
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const int col0 = half * 64 + cb * 32;
                    ptx::tmem_ld_32x32(lane_base + C::H_COL0 + buf * 128 + col0, r);
                    ptx::tmem_ld_wait();
                    const uint32_t hrow = hs + buf * kHBytes + (col0 >> 6) * 16384 + row * 128;
                    const int cc0 = (col0 & 63) >> 3;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t p[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            p[q] = pack_bf16x2(gelu_erf(__uint_as_float(r[8 * j + 2 * q])),
                                               gelu_erf(__uint_as_float(r[8 * j + 2 * q + 1])));
                        const uint32_t dst = hrow + (((cc0 + j) ^ (row & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(p[0]),
                                     "r"(p[1]), "r"(p[2]), "r"(p[3])
                                     : "memory");
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::fence_proxy_async_smem();
                ptx::mbar_arrive(ptx::smem_u32(&misc->h_tmem_empty[buf]));
                ptx::mbar_arrive(ptx::smem_u32(&misc->hs_full[buf]));
            }
            if (!ok) break;
            if (!ptx::mbar_wait(ptx::smem_u32(&misc->y_full), ti & 1u, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after_sync();
#pragma unroll 1
            for (int cb = 0; cb < D / 64; ++cb) {
                const int col0 = half * (D / 2) + cb * 32;
                ptx::tmem_ld_32x32(lane_base + col0, r);
                ptx::tmem_ld_wait();
                if (my_row >= 0) {
                    uint4* dst = reinterpret_cast<uint4*>(Y + (size_t)my_row * D + col0);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(r[8 * j]), __uint_as_float(r[8 * j + 1]));
                        v.y = pack_bf16x2(__uint_as_float(r[8 * j + 2]), __uint_as_float(r[8 * j + 3]));
                        v.z = pack_bf16x2(__uint_as_float(r[8 * j + 4]), __uint_as_float(r[8 * j + 5]));
                        v.w = pack_bf16x2(__uint_as_float(r[8 * j + 6]), __uint_as_float(r[8 * j + 7]));
                        dst[j] = v;
                    }
                }
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(ptx::smem_u32(&misc->y_empty));
            hc += NC;
        }
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
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 row-major [rows, cols] -> map with a 128-row x 64-column box, 128-byte swizzle.
bool make_weight_map(CUtensorMap* tm, void* ptr, uint64_t rows, uint64_t cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
int launch_d(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, const CUtensorMap& m1,
             const CUtensorMap& m2, int kc_pad, int max_tiles, cudaStream_t st) {
    auto kern = ffn_tc_kernel<D>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::SMEM_BYTES));
    int grid = max_tiles < ctx->sm_count ? max_tiles : ctx->sm_count;
    if (grid < 1) grid = 1;
    LaunchScope ls(ctx, KS_FFN_MAIN, st);
    kern<<<grid, kThreads, Cfg<D>::SMEM_BYTES, st>>>(m1, m2, (const __nv_bfloat16*)a.X, (__nv_bfloat16*)a.Y,
                                                      plan, a.d.n_lists, a.d.T, kc_pad, a.status);
    return SENTRY_OK;
}

}  // namespace

bool ffn_tc_supported(const sentry_ffn_desc& d) {
    return d.dtype == SENTRY_BF16 && (d.D == 128 || d.D == 256 || d.D == 384);
}

int ffn_tc_kc_pad(int k_c) { return (k_c + kChunk - 1) / kChunk * kChunk; }

int launch_ffn_tc(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c,
                  int kc_pad, int max_tiles, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    CUtensorMap m1, m2;
    if (!make_weight_map(&m1, w1c, (uint64_t)d.n_lists * kc_pad, (uint64_t)d.D)) return SENTRY_ERR_CUDA;
    if (!make_weight_map(&m2, w2c, (uint64_t)d.n_lists * d.D, (uint64_t)kc_pad)) return SENTRY_ERR_CUDA;
    int rc;
    switch (d.D) {
        case 128: rc = launch_d<128>(ctx, a, plan, m1, m2, kc_pad, max_tiles, st); break;
        case 256: rc = launch_d<256>(ctx, a, plan, m1, m2, kc_pad, max_tiles, st); break;
        case 384: rc = launch_d<384>(ctx, a, plan, m1, m2, kc_pad, max_tiles, st); break;
        default: return SENTRY_ERR_UNSUPPORTED;
    }
    if (rc != SENTRY_OK) return rc;
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

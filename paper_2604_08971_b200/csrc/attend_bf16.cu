// SentryAttend (Section 4.4, Eq. 6) for bf16 tensors: the fast path.
//
// Two kernels per call:
//   score  one CTA per (sample, KV group, 256 query positions).  The group's present K rows are
//          staged once in shared memory (16-byte async copies, XOR-swizzled rows); each thread
//          owns one query position and scores it against its sampled keys for ALL kept heads of
//          the group at once, so a sampled key row is fetched from shared memory once per group,
//          not once per head.       M_i = max_j s_ij - mean_j s_ij   (fp32)
//   core   one CTA per (sample, KV group).  Prologue: top-U selection per kept head (warp-level
//          threshold search on order-preserving keys; ties -> lower index).  Main loop: K/V tiles
//          of 64 present keys stream through shared memory once per GROUP and are shared by the
//          kept heads; the U active rows of each head run  softmax(q K^T / sqrt d) V  on the
//          warp-level tensor-core MMA with an online softmax (fp32 state in registers).  The
//          column sums of V ride along and give the context vector.  Epilogue: active rows,
//          context rows (mean of V_g) and zero rows (absent modalities) are written with
//          16-byte stores.  Pruned heads and unreferenced KV groups are never touched.
//
// The contraction here is tiny (U <= 45 rows per head against T_v keys): the path is bound by
// shared-memory gathers and HBM traffic, not by tensor throughput, which is why it uses the
// register-resident warp MMA rather than TMEM accumulators.
#include <math.h>

#include "attend_common.cuh"

namespace {




// Score pass for sequences whose K does not fit in shared memory at once: the group's present
// K rows pass through shared memory in segments of seg_rows (a power of two).  Each thread owns
// one query; it first sorts its sampled keys by segment into a per-thread list in shared memory
// (counting sort, counts packed in one 64-bit register), so that during a segment every lane
// walks only its own keys of that segment instead of skipping through the whole list.
template <int D, int NH>
__device__ __forceinline__ void long_score_pass(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ Kg,
                                                const uint16_t* s_valid, uint16_t* s_list, uint32_t ks_addr,
                                                int seg_shift, int Tv, int Tlen, const size_t* q_base,
                                                const int* khs, const int32_t* tbl_row, size_t tbl_es, int cnt,
                                                int score_mode, int p, int b, int k_h,
                                                float* __restrict__ mscore, unsigned int* status) {
    using S = Sw<D>;
    const bool act = p < Tv;
    const int seg_rows = 1 << seg_shift;
    uint32_t qw[NH][D / 2];
    float mx[NH], sum[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) { mx[h] = -INFINITY; sum[h] = 0.f; }
    unsigned long long starts = 0ull;   // byte s = first list slot of segment s (8 segments at most)
    if (act) {
        const int tok = s_valid[p];
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const uint4* src = reinterpret_cast<const uint4*>(Q + q_base[h] + (size_t)tok * D);
#pragma unroll
            for (int cc = 0; cc < S::CPR; ++cc) {
                const uint4 v = __ldg(src + cc);
                qw[h][4 * cc] = v.x; qw[h][4 * cc + 1] = v.y; qw[h][4 * cc + 2] = v.z; qw[h][4 * cc + 3] = v.w;
            }
        }
        if (score_mode != 1) {
            unsigned long long counts = 0ull;
            for (int a = 0; a < cnt; ++a) {
                int pj = __ldg(tbl_row + (size_t)a * tbl_es);
                if (pj < 0 || pj >= Tv) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); pj = 0; }
                counts += 1ull << (8 * (pj >> seg_shift));
            }
            unsigned long long run = 0ull;
#pragma unroll
            for (int sgm = 0; sgm < 8; ++sgm) {
                starts |= run << (8 * sgm);
                run += (counts >> (8 * sgm)) & 255ull;
            }
            unsigned long long fill = starts;
            for (int a = 0; a < cnt; ++a) {
                int pj = __ldg(tbl_row + (size_t)a * tbl_es);
                if (pj < 0 || pj >= Tv) pj = 0;
                const int sgm = pj >> seg_shift;
                const int pos = (int)((fill >> (8 * sgm)) & 255ull);
                fill += 1ull << (8 * sgm);
                s_list[pos * blockDim.x + threadIdx.x] = (uint16_t)pj;
            }
        }
    }
    const float scale = rsqrtf((float)D);
    int sgm = 0;
    for (int seg0 = 0; seg0 < Tv; seg0 += seg_rows, ++sgm) {
        const int seg_n = min(seg_rows, Tv - seg0);
        __syncthreads();  // the previous segment is no longer being read
        for (int i = threadIdx.x; i < seg_n * S::CPR; i += blockDim.x) {
            const int row = i / S::CPR, c = i % S::CPR;
            ptx::cp_async_16(ks_addr + S::off(row, c), Kg + (size_t)s_valid[seg0 + row] * D + c * 8);
        }
        ptx::cp_async_wait_all();
        __syncthreads();
        if (!act) continue;
        if (score_mode != 1) {
            const int i0 = (int)((starts >> (8 * sgm)) & 255ull);
            const int i1 = sgm == 7 ? cnt : (seg0 + seg_rows >= Tv ? cnt : (int)((starts >> (8 * (sgm + 1))) & 255ull));
            for (int i = i0; i < i1; ++i) {
                const int pj = s_list[i * blockDim.x + threadIdx.x];
                score_one_key<D, NH>(qw, ks_addr, pj - seg0, scale, mx, sum);
            }
        } else {
            for (int row = 0; row < seg_n; ++row) score_one_key<D, NH>(qw, ks_addr, row, scale, mx, sum);
        }
    }
    if (act) {
#pragma unroll
        for (int h = 0; h < NH; ++h)
            mscore[((size_t)b * k_h + khs[h]) * Tlen + p] = mx[h] - sum[h] / (float)cnt;
    }
}

// grid (B*Hk, ceil(T/threads)).  Dynamic smem: valid list (2T bytes, 128-aligned) | per-thread key
// lists [kMaxActive][threads] u16 | K segment.
template <int D>
__global__ void __launch_bounds__(kScoreThreads, 2)
attend_score_bf16_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                         const int32_t* __restrict__ kept_heads, const int32_t* __restrict__ ids,
                         const uint32_t* __restrict__ masks, const int32_t* __restrict__ table,
                         const int64_t* __restrict__ offsets, int n_subsets, int Tlen, int Hq, int Hk,
                         int k_h, int c, int score_mode, int seg_shift, float* __restrict__ mscore,
                         unsigned int* status) {
    extern __shared__ __align__(128) uint8_t s_raw[];
    __shared__ int red[66];
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(s_raw);
    const size_t valid_bytes = (((size_t)Tlen * 2 + 127) / 128) * 128;
    uint16_t* s_list = reinterpret_cast<uint16_t*>(s_raw + valid_bytes);
    const uint32_t ks_addr = ptx::smem_u32(s_raw) + (uint32_t)(valid_bytes + (size_t)kMaxActive * kScoreThreads * 2);
    const int b = blockIdx.x / Hk, g = blockIdx.x % Hk;
    const uint32_t mask = masks[b];
    const int Tv = block_build_valid(ids, Tlen, mask, s_valid, red);
    if (Tv == 0 || (int)(blockIdx.y * blockDim.x) >= Tv) return;
    int hs[kMaxRK], khs[kMaxRK];
    bool bad;
    const int rk = group_heads(kept_heads + (size_t)b * k_h, k_h, Hq / Hk, g, Hq, hs, khs, bad);
    if (bad && threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
    if (rk == 0) return;
    const int n_s = sentry_num_active(Tv, c);
    const int cnt = score_mode != 1 ? n_s : Tv;
    const int p = blockIdx.y * blockDim.x + threadIdx.x;
    const int32_t* tbl_row = nullptr;
    const size_t tbl_es = score_mode == 2 ? (size_t)Tv : 1;   // entry-major table: entry a of row p at a * Tv + p
    if (score_mode != 1) {
        if (mask >= (uint32_t)n_subsets || offsets[mask] < 0) {
            if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            return;
        }
        tbl_row = table + offsets[mask] + (size_t)min(p, Tv - 1) * (score_mode == 2 ? 1 : n_s);
    }
    const __nv_bfloat16* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    constexpr int HPP = (D == 64) ? 1 : (D == 32 ? 2 : 4);   // heads per pass: packed q rows live in registers
    for (int h0 = 0; h0 < rk; h0 += HPP) {
        const int nh = min(HPP, rk - h0);
        size_t q_base[4];
        int khs_[4];
        for (int j = 0; j < 4; ++j) {
            const int hh = min(h0 + j, rk - 1);
            q_base[j] = ((size_t)b * Hq + hs[hh]) * Tlen * D;
            khs_[j] = khs[hh];
        }
#define LONG_PASS(N) long_score_pass<D, N>(Q, Kg, s_valid, s_list, ks_addr, seg_shift, Tv, Tlen, q_base, khs_, \
                                           tbl_row, tbl_es, cnt, score_mode, p, b, k_h, mscore, status)
        if (nh == 1) LONG_PASS(1);
        else if (nh == 2) LONG_PASS(2);
        else if constexpr (HPP == 4) {
            if (nh == 3) LONG_PASS(3);
            else LONG_PASS(4);
        }
#undef LONG_PASS
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------- core
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32." ATT_PTX_TYPE "." ATT_PTX_TYPE ".f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];"
                 : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}


template <int D>
struct CoreSmem {
    static constexpr int TILE_BYTES = kKeyTile * D * 2;      // one K or V tile
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;       // K + V
    static constexpr int PIPE_BYTES = 2 * STAGE_BYTES;       // double buffered
};

// grid B*Hk.  Dynamic smem: valid[T] u16 | kind[T] u8 | actbits[4][T/32] u32 | union{keys, KV pipe}
template <int D>
__global__ void __launch_bounds__(kCoreThreads, 2)
attend_core_bf16_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                        const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ kept_heads,
                        const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks,
                        const float* __restrict__ mscore, const int32_t* __restrict__ active_in,
                        int32_t* __restrict__ active_out, int Tlen, int Hq, int Hk, int k_h, int c,
                        int U_max, __nv_bfloat16* __restrict__ O, unsigned int* status) {
    using S = Sw<D>;
    using CS = CoreSmem<D>;
    constexpr int NT = D / 8;        // n-tiles of the output (8 dims each)
    constexpr int KS = D / 16;       // k-steps of q.k
    extern __shared__ __align__(128) uint8_t s_raw[];
    __shared__ int red[66];
    __shared__ int32_t s_act[kMaxRK][kMaxActive];
    __shared__ float s_vpart[kCoreThreads / (D / 2)][D];   // partial column sums of V
    __shared__ int s_hist[kMaxRK][256];                    // radix-selection histograms, one per head
    __shared__ __align__(16) __nv_bfloat16 s_mean[D];

    const int words = (Tlen + 31) / 32;
    size_t o = 0;
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(s_raw + o); o += (((size_t)Tlen * 2 + 127) / 128) * 128;
    uint8_t* s_kind = s_raw + o;                                o += (((size_t)Tlen + 127) / 128) * 128;
    uint32_t* s_abits = reinterpret_cast<uint32_t*>(s_raw + o); o += (((size_t)kMaxRK * words * 4 + 127) / 128) * 128;
    uint8_t* s_union = s_raw + o;
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_union);
    const uint32_t pipe_addr = ptx::smem_u32(s_union);

    const int b = blockIdx.x / Hk, g = blockIdx.x % Hk;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int Tv = block_build_valid(ids, Tlen, masks[b], s_valid, red);
    int hs[kMaxRK], khs[kMaxRK];
    bool bad;
    const int rk = group_heads(kept_heads + (size_t)b * k_h, k_h, Hq / Hk, g, Hq, hs, khs, bad);
    if (rk == 0) return;
    if (Tv == 0) {  // no modality present: zero rows, flag
        for (int hh = 0; hh < rk; ++hh) {
            uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D);
            for (int i = threadIdx.x; i < Tlen * S::CPR; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
            if (active_out != nullptr && active_in == nullptr)
                for (int i = threadIdx.x; i < U_max; i += blockDim.x)
                    active_out[((size_t)b * k_h + khs[hh]) * U_max + i] = -1;
        }
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_EMPTY_MASK);
        return;
    }
    const int U = sentry_num_active(Tv, c);

    for (int t = threadIdx.x; t < Tlen; t += blockDim.x) s_kind[t] = 0;
    for (int i = threadIdx.x; i < kMaxRK * words; i += blockDim.x) s_abits[i] = 0u;
    for (int i = threadIdx.x; i < kMaxRK * kMaxActive; i += blockDim.x) (&s_act[0][0])[i] = -1;
    __syncthreads();
    for (int p = threadIdx.x; p < Tv; p += blockDim.x) s_kind[s_valid[p]] = 1;

    // ---- selection of the active rows (Section 4.4: the U queries with the largest score)
    if (active_in == nullptr) {
        for (int hh = 0; hh < rk; ++hh) {
            const float* m = mscore + ((size_t)b * k_h + khs[hh]) * Tlen;
            for (int p = threadIdx.x; p < Tv; p += blockDim.x) s_keys[(size_t)hh * Tv + p] = sentry_order_key(m[p]);
        }
        __syncthreads();
        if (warp < rk) warp_select_topk_radix(s_keys + (size_t)warp * Tv, Tv, U, s_act[warp], s_valid, s_hist[warp]);
        __syncthreads();
        if (active_out != nullptr)
            for (int i = threadIdx.x; i < rk * U_max; i += blockDim.x) {
                const int hh = i / U_max, a = i % U_max;
                active_out[((size_t)b * k_h + khs[hh]) * U_max + a] = a < U ? s_act[hh][a] : -1;
            }
    } else {
        __syncthreads();
        for (int i = threadIdx.x; i < rk * kMaxActive; i += blockDim.x) {
            const int hh = i / kMaxActive, a = i % kMaxActive;
            int t = a < U_max ? active_in[((size_t)b * k_h + khs[hh]) * U_max + a] : -1;
            if (t >= 0 && (t >= Tlen || s_kind[t] == 0)) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); t = -1; }
            s_act[hh][a] = t;
        }
        __syncthreads();
    }
    for (int i = threadIdx.x; i < rk * kMaxActive; i += blockDim.x) {
        const int hh = i / kMaxActive, t = s_act[hh][i % kMaxActive];
        if (t >= 0) atomicOr(&s_abits[hh * words + (t >> 5)], 1u << (t & 31));
    }
    __syncthreads();   // s_keys is dead from here on: the union becomes the K/V pipe

    // ---- row tiles of this warp: tile tt -> (head slot, 16 active rows)
    const int WT = (min(U, kMaxActive) + 15) / 16;     // row tiles per head (<= 3)
    const int n_tiles = rk * WT;
    const int gq = lane >> 2, tq = lane & 3;
    uint32_t qf[2][KS][4];
    float acc[2][NT][4];
    float m_run[2][2], l_run[2][2];
    int tile_head[2], tile_row0[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int tt = warp + j * kCoreWarps;
        tile_head[j] = tt < n_tiles ? tt / WT : -1;
        tile_row0[j] = tt < n_tiles ? (tt % WT) * 16 : 0;
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[j][n][e] = 0.f;
        m_run[j][0] = m_run[j][1] = -INFINITY;
        l_run[j][0] = l_run[j][1] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int e = 0; e < 4; ++e) qf[j][ks][e] = 0u;
        if (tile_head[j] >= 0) {
            const int hh = tile_head[j];
            const __nv_bfloat16* Qh = Q + ((size_t)b * Hq + hs[hh]) * Tlen * D;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int a = tile_row0[j] + gq + half * 8;
                const int t = a < kMaxActive ? s_act[hh][a] : -1;
                if (t >= 0) {
                    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(Qh + (size_t)t * D);
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        qf[j][ks][half] = __ldg(qrow + ks * 8 + tq);          // cols 16ks + 2t, +1
                        qf[j][ks][half + 2] = __ldg(qrow + ks * 8 + 4 + tq);  // cols 16ks + 8 + 2t, +1
                    }
                }
            }
        }
    }

    // ---- stream K/V tiles of 64 present keys
    const __nv_bfloat16* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    const __nv_bfloat16* Vg = V + ((size_t)b * Hk + g) * Tlen * D;
    const int n_kt = (Tv + kKeyTile - 1) / kKeyTile;
    auto load_tile = [&](int kt, int stage) {
        const uint32_t kbase = pipe_addr + stage * CS::STAGE_BYTES;
        const uint32_t vbase = kbase + CS::TILE_BYTES;
        const int rows = min(kKeyTile, Tv - kt * kKeyTile);
        for (int i = threadIdx.x; i < kKeyTile * S::CPR; i += blockDim.x) {
            const int row = i / S::CPR, cc = i % S::CPR;
            if (row < rows) {
                const size_t goff = (size_t)s_valid[kt * kKeyTile + row] * D + cc * 8;
                ptx::cp_async_16(kbase + S::off(row, cc), Kg + goff);
                ptx::cp_async_16(vbase + S::off(row, cc), Vg + goff);
            } else {  // keys past the end: zeros (masked out of the softmax, add nothing to sums)
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(kbase + S::off(row, cc)), "r"(0) : "memory");
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vbase + S::off(row, cc)), "r"(0) : "memory");
            }
        }
        ptx::cp_async_commit();
    };
    // V column sums: thread -> (dim pair, key residue)
    constexpr int DP = D / 2;
    const int vs_dp = threadIdx.x % DP, vs_k0 = threadIdx.x / DP;
    constexpr int VS_STRIDE = kCoreThreads / DP;
    float vsum0 = 0.f, vsum1 = 0.f;

    const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;  // scale * log2(e)
    load_tile(0, 0);
    for (int kt = 0; kt < n_kt; ++kt) {
        const int stage = kt & 1;
        if (kt + 1 < n_kt) { load_tile(kt + 1, stage ^ 1); ptx::cp_async_wait_group<1>(); }
        else ptx::cp_async_wait_group<0>();
        __syncthreads();
        const uint32_t kbase = pipe_addr + stage * CS::STAGE_BYTES;
        const uint32_t vbase = kbase + CS::TILE_BYTES;
        const int key0 = kt * kKeyTile;
        // column sums of V (padding rows are zero)
        for (int row = vs_k0; row < kKeyTile; row += VS_STRIDE) {
            uint32_t w;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(vbase + S::off(row, vs_dp >> 2) + (vs_dp & 3) * 4));
            vsum0 += att_lo(w);
            vsum1 += att_hi(w);
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (tile_head[j] < 0) continue;   // warp-uniform
            // S = q K^T for 16 rows x 64 keys
            float s[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
                const int krow = nt * 8 + (lane & 7);
                if constexpr (D == 32) {
                    uint32_t bfr[4];
                    ldmatrix_x4(kbase + S::off(krow, lane >> 3), bfr);
                    mma_bf16_16816(s[nt], qf[j][0], bfr[0], bfr[1]);
                    mma_bf16_16816(s[nt], qf[j][1], bfr[2], bfr[3]);
                } else if constexpr (D == 16) {
                    uint32_t bfr[2];
                    ldmatrix_x2(kbase + S::off(krow, (lane >> 3) & 1), bfr);
                    mma_bf16_16816(s[nt], qf[j][0], bfr[0], bfr[1]);
                } else {  // D == 64
                    uint32_t bfr[4];
                    ldmatrix_x4(kbase + S::off(krow, lane >> 3), bfr);
                    mma_bf16_16816(s[nt], qf[j][0], bfr[0], bfr[1]);
                    mma_bf16_16816(s[nt], qf[j][1], bfr[2], bfr[3]);
                    ldmatrix_x4(kbase + S::off(krow, 4 + (lane >> 3)), bfr);
                    mma_bf16_16816(s[nt], qf[j][2], bfr[0], bfr[1]);
                    mma_bf16_16816(s[nt], qf[j][3], bfr[2], bfr[3]);
                }
            }
            // online softmax over this tile (rows gq and gq+8), base-2 exponent
            float mt[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = key0 + nt * 8 + tq * 2 + (e & 1);
                    s[nt][e] = key < Tv ? s[nt][e] * sl2 : -INFINITY;
                    mt[e >> 1] = fmaxf(mt[e >> 1], s[nt][e]);
                }
            float corr[2];
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                mt[h2] = fmaxf(mt[h2], __shfl_xor_sync(0xffffffffu, mt[h2], 1));
                mt[h2] = fmaxf(mt[h2], __shfl_xor_sync(0xffffffffu, mt[h2], 2));
                const float m_new = fmaxf(m_run[j][h2], mt[h2]);
                corr[h2] = fast_exp2(m_run[j][h2] - m_new);   // 0 on the first tile
                m_run[j][h2] = m_new;
                l_run[j][h2] *= corr[h2];
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) s[nt][e] = fast_exp2(s[nt][e] - m_run[j][e >> 1]);
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                acc[j][n][0] *= corr[0]; acc[j][n][1] *= corr[0];
                acc[j][n][2] *= corr[1]; acc[j][n][3] *= corr[1];
            }
            // O += P V
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t pa[4];
                pa[0] = pack2(s[2 * ks][0], s[2 * ks][1]);
                pa[1] = pack2(s[2 * ks][2], s[2 * ks][3]);
                pa[2] = pack2(s[2 * ks + 1][0], s[2 * ks + 1][1]);
                pa[3] = pack2(s[2 * ks + 1][2], s[2 * ks + 1][3]);
                // every weight goes to the tensor core as a bf16 head plus a bf16 remainder
                // (p = p_hi + p_lo to 2^-17), so the rounding of the weights drops out of O
                uint32_t pb[4];
                pb[0] = pack2_rem(s[2 * ks][0], s[2 * ks][1], pa[0]);
                pb[1] = pack2_rem(s[2 * ks][2], s[2 * ks][3], pa[1]);
                pb[2] = pack2_rem(s[2 * ks + 1][0], s[2 * ks + 1][1], pa[2]);
                pb[3] = pack2_rem(s[2 * ks + 1][2], s[2 * ks + 1][3], pa[3]);
                l_run[j][0] += (s[2 * ks][0] + s[2 * ks][1]) + (s[2 * ks + 1][0] + s[2 * ks + 1][1]);
                l_run[j][1] += (s[2 * ks][2] + s[2 * ks][3]) + (s[2 * ks + 1][2] + s[2 * ks + 1][3]);
                const int vrow = ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                for (int n2 = 0; n2 < NT / 2; ++n2) {
                    uint32_t bfr[4];
                    ldmatrix_x4_trans(vbase + S::off(vrow, 2 * n2 + (lane >> 4)), bfr);
                    mma_bf16_16816(acc[j][2 * n2], pa, bfr[0], bfr[1]);
                    mma_bf16_16816(acc[j][2 * n2 + 1], pa, bfr[2], bfr[3]);
                    mma_bf16_16816(acc[j][2 * n2], pb, bfr[0], bfr[1]);
                    mma_bf16_16816(acc[j][2 * n2 + 1], pb, bfr[2], bfr[3]);
                }
            }
        }
        __syncthreads();   // everyone is done with this stage before it is refilled
    }

    // ---- context vector = mean of V_g over the present keys
    s_vpart[vs_k0][2 * vs_dp] = vsum0;
    s_vpart[vs_k0][2 * vs_dp + 1] = vsum1;
    __syncthreads();
    if (threadIdx.x < D) {
        float t = 0.f;
        for (int i = 0; i < VS_STRIDE; ++i) t += s_vpart[i][threadIdx.x];
        reinterpret_cast<unsigned short*>(s_mean)[threadIdx.x] = att_bits(t / (float)Tv);
    }
    // ---- active rows: normalise and store
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        if (tile_head[j] < 0) continue;
        const int hh = tile_head[j];
        __nv_bfloat16* Oh = O + ((size_t)b * k_h + khs[hh]) * Tlen * D;
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            float l = l_run[j][h2];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int a = tile_row0[j] + gq + h2 * 8;
            const int t = a < kMaxActive ? s_act[hh][a] : -1;
            if (t < 0) continue;
            const float inv = 1.0f / l;
            uint32_t* orow = reinterpret_cast<uint32_t*>(Oh + (size_t)t * D);
#pragma unroll
            for (int n = 0; n < NT; ++n)
                orow[n * 4 + tq] = pack2(acc[j][n][2 * h2] * inv, acc[j][n][2 * h2 + 1] * inv);
        }
    }
    __syncthreads();
    // ---- context rows and zero rows, 16 bytes per store
    const uint4* mean4 = reinterpret_cast<const uint4*>(s_mean);
    for (int hh = 0; hh < rk; ++hh) {
        uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D);
        const uint32_t* bits = s_abits + hh * words;
        for (int i = threadIdx.x; i < Tlen * S::CPR; i += blockDim.x) {
            const int t = i / S::CPR, cc = i % S::CPR;
            if ((bits[t >> 5] >> (t & 31)) & 1u) continue;
            dst[i] = s_kind[t] ? mean4[cc] : make_uint4(0, 0, 0, 0);
        }
    }
}

// ------------------------------------------------------------------------------------ fused
// One CTA per (sample, KV group) does the whole of SentryAttend for the group's kept heads
// when the group's present K and V rows fit in shared memory (T up to ~1.5 k at d = 32):
//   stage K, V (gathered present rows, once) -> sparsity scores from shared memory ->
//   top-U per head (one warp per head, radix selection) -> Eq. 6 on the active rows with the
//   warp-level tensor-core MMA straight from the resident K/V -> context rows and zero rows.
// Q, K, V are read from HBM once and O is written once: the algorithmic traffic.

// Sparsity scores of NH heads of the group at once for the queries of this thread:
// M_i = max_j s_ij - mean_j s_ij over the sampled (or all) present keys, K rows from shared
// memory.  The order keys of the scores go to keys_out[h][p].  The query rows stay in
// registers as packed bf16 (D/2 words per head), so all kept heads of a group fit in one pass
// and a sampled key row is fetched once per group.
template <int D, int NH>
__device__ __forceinline__ void fused_score_pass(const __nv_bfloat16* __restrict__ Q,
                                                 const size_t* q_base, const uint16_t* s_valid,
                                                 uint32_t ks_addr, int Tv,
                                                 const int32_t* __restrict__ tbl, int n_s, int cnt,
                                                 int score_mode, uint32_t* const* keys_out,
                                                 unsigned int* status) {
    using S = Sw<D>;
    const float scale = rsqrtf((float)D);
    const float inv_cnt = 1.0f / (float)cnt;
    for (int p = threadIdx.x; p < Tv; p += blockDim.x) {
        const int tok = s_valid[p];
        uint32_t qw[NH][D / 2];
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const uint4* src = reinterpret_cast<const uint4*>(Q + q_base[h] + (size_t)tok * D);
#pragma unroll
            for (int cc = 0; cc < S::CPR; ++cc) {
                const uint4 v = __ldg(src + cc);
                qw[h][4 * cc] = v.x; qw[h][4 * cc + 1] = v.y; qw[h][4 * cc + 2] = v.z; qw[h][4 * cc + 3] = v.w;
            }
        }
        float mx[NH], sum[NH];
#pragma unroll
        for (int h = 0; h < NH; ++h) { mx[h] = -INFINITY; sum[h] = 0.f; }
        // The sampled positions come four at a time, the next four requested before the current
        // four are used: a thread walks its own table row, and with most of the L1 given to
        // shared memory the row's lines do not survive from one use to the next.
        // query-major table: entry a of row p at p * n_s + a; entry-major (score_mode 2): a * Tv + p
        const int32_t* row = score_mode != 1 ? tbl + (size_t)p * (score_mode == 2 ? 1 : n_s) : nullptr;
        const size_t es = score_mode == 2 ? (size_t)Tv : 1;
        int nxt[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) nxt[u] = score_mode != 1 ? __ldg(row + (size_t)min(u, cnt - 1) * es) : u;
        for (int a0 = 0; a0 < cnt; a0 += 4) {
            int cur[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                cur[u] = nxt[u];
                nxt[u] = score_mode != 1 ? __ldg(row + (size_t)min(a0 + 4 + u, cnt - 1) * es) : a0 + 4 + u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (a0 + u >= cnt) break;
                int pj = cur[u];
                if (pj < 0 || pj >= Tv) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); pj = 0; }
                float acc[NH][4];
#pragma unroll
                for (int h = 0; h < NH; ++h) acc[h][0] = acc[h][1] = acc[h][2] = acc[h][3] = 0.f;
#pragma unroll
                for (int cc = 0; cc < S::CPR; ++cc) {
                    const uint4 v = lds128(ks_addr + S::off(pj, cc));
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        fma_bf16_pair(acc[h][0], acc[h][1], qw[h][4 * cc], v.x);
                        fma_bf16_pair(acc[h][2], acc[h][3], qw[h][4 * cc + 1], v.y);
                        fma_bf16_pair(acc[h][0], acc[h][1], qw[h][4 * cc + 2], v.z);
                        fma_bf16_pair(acc[h][2], acc[h][3], qw[h][4 * cc + 3], v.w);
                    }
                }
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    const float sc = ((acc[h][0] + acc[h][1]) + (acc[h][2] + acc[h][3])) * scale;
                    mx[h] = fmaxf(mx[h], sc);
                    sum[h] += sc;
                }
            }
        }
#pragma unroll
        for (int h = 0; h < NH; ++h) keys_out[h][p] = sentry_order_key(mx[h] - sum[h] * inv_cnt);
    }
}

// grid B*Hk, 256 or 512 threads.  Dynamic smem: valid[T] u16 | kind[T] u8 | actbits[4][T/32] u32 |
// keys[4][T] u32 | hist[4][256] | K[Tpad][D] | V[Tpad][D]   (Tpad = T rounded up to 64).
template <int D>
__global__ void __launch_bounds__(512, 1)
attend_fused_bf16_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                         const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ kept_heads,
                         const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks,
                         const int32_t* __restrict__ table, const int64_t* __restrict__ offsets,
                         int n_subsets, const int32_t* __restrict__ active_in,
                         int32_t* __restrict__ active_out, int Tlen, int Hq, int Hk, int k_h, int c,
                         int score_mode, int U_max, __nv_bfloat16* __restrict__ O, unsigned int* status,
                         const float* __restrict__ gate_scores, int gate_S, int32_t* __restrict__ kept_out) {
    using S = Sw<D>;
    constexpr int NT = D / 8;        // n-tiles of the output (8 dims each)
    constexpr int KS = D / 16;       // k-steps of q.k
    constexpr int TILE_BYTES = kKeyTile * D * 2;
    extern __shared__ __align__(128) uint8_t s_raw[];
    __shared__ int red[66];
    __shared__ int32_t s_kept[64];
    __shared__ int32_t s_act[kMaxRK][kMaxActive];
    __shared__ float s_vpart[512 / (D / 2)][D];
    __shared__ __align__(16) __nv_bfloat16 s_mean[D];

    const int words = (Tlen + 31) / 32;
    const int Tpad = (Tlen + kKeyTile - 1) / kKeyTile * kKeyTile;
    size_t o = 0;
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(s_raw + o); o += (((size_t)Tlen * 2 + 127) / 128) * 128;
    uint8_t* s_kind = s_raw + o;                                o += (((size_t)Tlen + 127) / 128) * 128;
    uint32_t* s_abits = reinterpret_cast<uint32_t*>(s_raw + o); o += (((size_t)kMaxRK * words * 4 + 127) / 128) * 128;
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_raw + o);  o += (((size_t)kMaxRK * Tlen * 4 + 127) / 128) * 128;
    int* s_hist = reinterpret_cast<int*>(s_raw + o);            o += (size_t)kMaxRK * 256 * 4;
    const uint32_t ks_addr = ptx::smem_u32(s_raw + o);          o += (size_t)Tpad * D * 2;
    const uint32_t vs_addr = ptx::smem_u32(s_raw + o);

    // Samples with more modalities present take longer; in small batches the CTAs take them
    // heaviest first (every CTA finds the sample of its rank by itself with a counting sort on
    // the number of present modalities), so that the long ones do not end up alone in the tail
    // of the launch.
    __shared__ int s_fill_next;
    if (threadIdx.x == 0) s_fill_next = 0;
    int b = blockIdx.x / Hk;
    const int g = blockIdx.x % Hk;
    const int Bn = gridDim.x / Hk;
    if (Bn > 1 && Bn <= kOrderMaxBatch) {
        __shared__ int s_cls[33];
        __shared__ int s_wcnt[16];
        __shared__ int s_pick[2];
        const int lane_ = threadIdx.x & 31, wid_ = threadIdx.x >> 5, nw_ = blockDim.x >> 5;
        if (threadIdx.x < 33) s_cls[threadIdx.x] = 0;
        __syncthreads();
        // samples per class (number of present modalities): one shared-memory atomic per warp and class
        for (int b0 = 0; b0 < Bn; b0 += blockDim.x) {
            const int bb = b0 + threadIdx.x;
            const int c = bb < Bn ? __popc(masks[bb]) : -1;
            const unsigned peers = __match_any_sync(0xffffffffu, c);
            if (c >= 0 && lane_ == __ffs(peers) - 1) atomicAdd(&s_cls[c], __popc(peers));
        }
        __syncthreads();
        // every warp for itself: the class that holds rank b, classes descending (lane l <-> class 32 - l;
        // what no lane claims is class 0), and the offset in it
        int cls, need;
        {
            const int mine = s_cls[32 - lane_];
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane_ >= o) incl += v;
            }
            const int above = incl - mine;
            const unsigned hit = __ballot_sync(0xffffffffu, above <= b && b < incl);
            const int src = hit ? __ffs(hit) - 1 : 31;
            const int above_src = __shfl_sync(0xffffffffu, above, src), incl_src = __shfl_sync(0xffffffffu, incl, src);
            cls = hit ? 32 - src : 0;
            need = hit ? b - above_src : b - incl_src;   // the need-th sample of that class, in index order
        }
        for (int b0 = 0; b0 < Bn; b0 += blockDim.x) {
            const int bb = b0 + threadIdx.x;
            const bool hit = bb < Bn && __popc(masks[bb]) == cls;
            const unsigned bm = __ballot_sync(0xffffffffu, hit);
            if (lane_ == 0) s_wcnt[wid_] = __popc(bm);
            __syncthreads();
            int before = 0, tot = 0;
            for (int w = 0; w < nw_; ++w) { if (w < wid_) before += s_wcnt[w]; tot += s_wcnt[w]; }
            if (hit && before + __popc(bm & ((1u << lane_) - 1u)) == need) s_pick[0] = bb;
            __syncthreads();
            if (need < tot) break;
            need -= tot;
        }
        b = s_pick[0];
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const uint32_t mask = masks[b];
    const int Tv = block_build_valid(ids, Tlen, mask, s_valid, red);
    const int32_t* kept_row = kept_heads + (size_t)b * k_h;
    if (gate_scores != nullptr) {
        // SentryGate's head selection for this sample's mask, done here instead of by a launch of
        // its own: the k_h best of the Hq <= 64 scores of row `mask` (score descending, equal
        // scores -> lower index, NaN below every number), ascending.  Every CTA of the sample
        // computes the same list; the CTA of group 0 leaves it in kept_out.
        if (warp == 0) {
            uint32_t row = mask;
            if (row >= (uint32_t)gate_S) { if (lane == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); row = 0; }
            const float* sr = gate_scores + (size_t)row * Hq;
            const uint32_t k0 = lane < Hq ? sentry_order_key(sr[lane]) : 0u;
            const uint32_t k1 = lane + 32 < Hq ? sentry_order_key(sr[lane + 32]) : 0u;
            int r0 = 0, r1 = 0;
            for (int j = 0; j < Hq; ++j) {
                const uint32_t kj = __shfl_sync(0xffffffffu, j < 32 ? k0 : k1, j & 31);
                r0 += (kj > k0 || (kj == k0 && j < lane)) ? 1 : 0;
                r1 += (kj > k1 || (kj == k1 && j < lane + 32)) ? 1 : 0;
            }
            const bool keep0 = lane < Hq && r0 < k_h, keep1 = lane + 32 < Hq && r1 < k_h;
            const unsigned b0 = __ballot_sync(0xffffffffu, keep0), b1 = __ballot_sync(0xffffffffu, keep1);
            const unsigned lt = (1u << lane) - 1u;
            if (keep0) s_kept[__popc(b0 & lt)] = lane;
            if (keep1) s_kept[__popc(b0) + __popc(b1 & lt)] = lane + 32;
        }
        __syncthreads();
        if (g == 0 && kept_out != nullptr && (int)threadIdx.x < k_h) kept_out[(size_t)b * k_h + threadIdx.x] = s_kept[threadIdx.x];
        kept_row = s_kept;
    }
    int hs[kMaxRK], khs[kMaxRK];
    bool bad;
    const int rk = group_heads(kept_row, k_h, Hq / Hk, g, Hq, hs, khs, bad);
    if (bad && threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
    if (rk == 0) return;
    if (Tv == 0) {  // no modality present: zero rows, flag
        for (int hh = 0; hh < rk; ++hh) {
            uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D);
            for (int i = threadIdx.x; i < Tlen * S::CPR; i += blockDim.x) dst[i] = make_uint4(0, 0, 0, 0);
            if (active_out != nullptr && active_in == nullptr)
                for (int i = threadIdx.x; i < U_max; i += blockDim.x)
                    active_out[((size_t)b * k_h + khs[hh]) * U_max + i] = -1;
        }
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_EMPTY_MASK);
        return;
    }
    const int U = sentry_num_active(Tv, c);

    // ---- stage the group's present K rows, then V rows (two copy groups), zero the padding
    const __nv_bfloat16* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    const __nv_bfloat16* Vg = V + ((size_t)b * Hk + g) * Tlen * D;
    const int n_kt = (Tv + kKeyTile - 1) / kKeyTile;
    const int rows_staged = n_kt * kKeyTile;
    for (int i = threadIdx.x; i < rows_staged * S::CPR; i += blockDim.x) {
        const int row = i / S::CPR, cc = i % S::CPR;
        if (row < Tv) ptx::cp_async_16(ks_addr + S::off(row, cc), Kg + (size_t)s_valid[row] * D + cc * 8);
        else asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(ks_addr + S::off(row, cc)), "r"(0) : "memory");
    }
    ptx::cp_async_commit();
    for (int i = threadIdx.x; i < rows_staged * S::CPR; i += blockDim.x) {
        const int row = i / S::CPR, cc = i % S::CPR;
        if (row < Tv) ptx::cp_async_16(vs_addr + S::off(row, cc), Vg + (size_t)s_valid[row] * D + cc * 8);
        else asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vs_addr + S::off(row, cc)), "r"(0) : "memory");
    }
    ptx::cp_async_commit();

    for (int t = threadIdx.x; t < Tlen; t += blockDim.x) s_kind[t] = 0;
    for (int i = threadIdx.x; i < kMaxRK * words; i += blockDim.x) s_abits[i] = 0u;
    for (int i = threadIdx.x; i < kMaxRK * kMaxActive; i += blockDim.x) (&s_act[0][0])[i] = -1;
    __syncthreads();
    for (int p = threadIdx.x; p < Tv; p += blockDim.x) s_kind[s_valid[p]] = 1;

    if (active_in == nullptr) {
        // ---- sparsity scores (Section 4.4) from the resident K rows
        const int n_s = U;
        const int cnt = score_mode != 1 ? n_s : Tv;
        const int32_t* tbl = nullptr;
        bool table_ok = true;
        if (score_mode != 1) {
            if (mask >= (uint32_t)n_subsets || offsets[mask] < 0) table_ok = false;
            else tbl = table + offsets[mask];
        }
        ptx::cp_async_wait_group<1>();   // K has landed (V may still be in flight)
        __syncthreads();
        if (table_ok) {
            constexpr int HPP = (D == 64) ? 2 : 4;   // heads per pass: packed q rows live in registers
            for (int h0 = 0; h0 < rk; h0 += HPP) {
                const int nh = min(HPP, rk - h0);
                size_t q_base[4];
                uint32_t* keys_out[4];
                for (int j = 0; j < 4; ++j) {
                    const int hh = min(h0 + j, rk - 1);
                    q_base[j] = ((size_t)b * Hq + hs[hh]) * Tlen * D;
                    keys_out[j] = s_keys + (size_t)hh * Tlen;
                }
                if (nh == 1) fused_score_pass<D, 1>(Q, q_base, s_valid, ks_addr, Tv, tbl, n_s, cnt, score_mode, keys_out, status);
                else if (nh == 2) fused_score_pass<D, 2>(Q, q_base, s_valid, ks_addr, Tv, tbl, n_s, cnt, score_mode, keys_out, status);
                else if constexpr (HPP == 4) {
                    if (nh == 3) fused_score_pass<D, 3>(Q, q_base, s_valid, ks_addr, Tv, tbl, n_s, cnt, score_mode, keys_out, status);
                    else fused_score_pass<D, 4>(Q, q_base, s_valid, ks_addr, Tv, tbl, n_s, cnt, score_mode, keys_out, status);
                }
            }
        } else {
            if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            for (int i = threadIdx.x; i < rk * Tlen; i += blockDim.x) s_keys[i] = 0u;
        }
        __syncthreads();
        // ---- the U present queries with the largest score are active
        // short lists: one warp per head with the keys in registers; longer ones: digit counting
        // by the whole block (measured: the warp form wins up to 256 keys, loses from 1024 on)
        if (Tv <= 256) warps_select_topk_heads(s_keys, Tlen, Tv, U, rk, s_act, s_valid);
        else block_select_topk_heads(s_keys, Tlen, Tv, U, rk, s_act, s_valid, s_hist);
        __syncthreads();
        if (active_out != nullptr)
            for (int i = threadIdx.x; i < rk * U_max; i += blockDim.x) {
                const int hh = i / U_max, a = i % U_max;
                active_out[((size_t)b * k_h + khs[hh]) * U_max + a] = a < U ? s_act[hh][a] : -1;
            }
    } else {
        __syncthreads();
        for (int i = threadIdx.x; i < rk * kMaxActive; i += blockDim.x) {
            const int hh = i / kMaxActive, a = i % kMaxActive;
            int t = a < U_max ? active_in[((size_t)b * k_h + khs[hh]) * U_max + a] : -1;
            if (t >= 0 && (t >= Tlen || s_kind[t] == 0)) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); t = -1; }
            s_act[hh][a] = t;
        }
        __syncthreads();
    }
    for (int i = threadIdx.x; i < rk * kMaxActive; i += blockDim.x) {
        const int hh = i / kMaxActive, t = s_act[hh][i % kMaxActive];
        if (t >= 0) atomicOr(&s_abits[hh * words + (t >> 5)], 1u << (t & 31));
    }
    ptx::cp_async_wait_group<0>();       // V has landed
    __syncthreads();

    // ---- context vector = mean of V_g over the present keys (padding rows are zero)
    {
        constexpr int DP = D / 2;
        const int vs_dp = threadIdx.x % DP, vs_k0 = threadIdx.x / DP;
        const int stride = blockDim.x / DP;
        float v0 = 0.f, v1 = 0.f;
        for (int row = vs_k0; row < rows_staged; row += stride) {
            uint32_t w;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(vs_addr + S::off(row, vs_dp >> 2) + (vs_dp & 3) * 4));
            v0 += att_lo(w);
            v1 += att_hi(w);
        }
        s_vpart[vs_k0][2 * vs_dp] = v0;
        s_vpart[vs_k0][2 * vs_dp + 1] = v1;
        __syncthreads();
        if (threadIdx.x < D) {
            float t = 0.f;
            for (int i = 0; i < stride; ++i) t += s_vpart[i][threadIdx.x];
            reinterpret_cast<unsigned short*>(s_mean)[threadIdx.x] = att_bits(t / (float)Tv);
        }
    }
    __syncthreads();   // s_mean is complete: warps without a row tile go straight to the fill

    // ---- Eq. 6 on the active rows: tiles of 16 rows over the warps.  The heads of a group share K
    // and V, so a tile may hold rows of several heads: the rk * U active rows are packed back to
    // back (U = 35: 7 tiles for three heads instead of 3 x 3, the last of each nearly empty).
    const int Ue = min(U, kMaxActive);
    const int n_rows_act = rk * Ue;
    const int n_tiles = (n_rows_act + 15) / 16;
    const int gq = lane >> 2, tq = lane & 3;
    const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;  // scale * log2(e)
    for (int tt = warp; tt < n_tiles; tt += nwarps) {
        // this lane's two rows (gq and gq + 8 of the tile): token, head, output head slot
        int row_t[2], row_kh[2];
        const __nv_bfloat16* row_q[2];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = tt * 16 + gq + half * 8;
            int hh = 0, t = -1;
            if (r < n_rows_act) {
                hh = r / Ue;
                t = s_act[hh][r - hh * Ue];
            }
            int h_sel = hs[0], kh_sel = khs[0];
#pragma unroll
            for (int j = 1; j < kMaxRK; ++j)
                if (hh == j) { h_sel = hs[j]; kh_sel = khs[j]; }
            row_t[half] = t;
            row_kh[half] = kh_sel;
            row_q[half] = Q + ((size_t)b * Hq + h_sel) * Tlen * D;
        }
        uint32_t qf[KS][4];
        float acc[NT][4];
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[n][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int e = 0; e < 4; ++e) qf[ks][e] = 0u;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int t = row_t[half];
            if (t >= 0) {
                const uint32_t* qrow = reinterpret_cast<const uint32_t*>(row_q[half] + (size_t)t * D);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    qf[ks][half] = __ldg(qrow + ks * 8 + tq);          // cols 16ks + 2t, +1
                    qf[ks][half + 2] = __ldg(qrow + ks * 8 + 4 + tq);  // cols 16ks + 8 + 2t, +1
                }
            }
        }
        for (int kt = 0; kt < n_kt; ++kt) {
            const uint32_t kbase = ks_addr + kt * TILE_BYTES;
            const uint32_t vbase = vs_addr + kt * TILE_BYTES;
            const int key0 = kt * kKeyTile;
            float sc[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) sc[nt][e] = 0.f;
                const int krow = nt * 8 + (lane & 7);
                if constexpr (D == 32) {
                    uint32_t bfr[4];
                    ldmatrix_x4(kbase + S::off(krow, lane >> 3), bfr);
                    mma_bf16_16816(sc[nt], qf[0], bfr[0], bfr[1]);
                    mma_bf16_16816(sc[nt], qf[1], bfr[2], bfr[3]);
                } else if constexpr (D == 16) {
                    uint32_t bfr[2];
                    ldmatrix_x2(kbase + S::off(krow, (lane >> 3) & 1), bfr);
                    mma_bf16_16816(sc[nt], qf[0], bfr[0], bfr[1]);
                } else {
                    uint32_t bfr[4];
                    ldmatrix_x4(kbase + S::off(krow, lane >> 3), bfr);
                    mma_bf16_16816(sc[nt], qf[0], bfr[0], bfr[1]);
                    mma_bf16_16816(sc[nt], qf[1], bfr[2], bfr[3]);
                    ldmatrix_x4(kbase + S::off(krow, 4 + (lane >> 3)), bfr);
                    mma_bf16_16816(sc[nt], qf[2], bfr[0], bfr[1]);
                    mma_bf16_16816(sc[nt], qf[3], bfr[2], bfr[3]);
                }
            }
            float mt[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = key0 + nt * 8 + tq * 2 + (e & 1);
                    sc[nt][e] = key < Tv ? sc[nt][e] * sl2 : -INFINITY;
                    mt[e >> 1] = fmaxf(mt[e >> 1], sc[nt][e]);
                }
            float corr[2];
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                mt[h2] = fmaxf(mt[h2], __shfl_xor_sync(0xffffffffu, mt[h2], 1));
                mt[h2] = fmaxf(mt[h2], __shfl_xor_sync(0xffffffffu, mt[h2], 2));
                const float m_new = fmaxf(m_run[h2], mt[h2]);
                corr[h2] = fast_exp2(m_run[h2] - m_new);   // 0 on the first tile
                m_run[h2] = m_new;
                l_run[h2] *= corr[h2];
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) sc[nt][e] = fast_exp2(sc[nt][e] - m_run[e >> 1]);
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                acc[n][0] *= corr[0]; acc[n][1] *= corr[0];
                acc[n][2] *= corr[1]; acc[n][3] *= corr[1];
            }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t pa[4];
                pa[0] = pack2(sc[2 * ks][0], sc[2 * ks][1]);
                pa[1] = pack2(sc[2 * ks][2], sc[2 * ks][3]);
                pa[2] = pack2(sc[2 * ks + 1][0], sc[2 * ks + 1][1]);
                pa[3] = pack2(sc[2 * ks + 1][2], sc[2 * ks + 1][3]);
                // bf16 head plus bf16 remainder of every weight (see the streamed kernel)
                uint32_t pb[4];
                pb[0] = pack2_rem(sc[2 * ks][0], sc[2 * ks][1], pa[0]);
                pb[1] = pack2_rem(sc[2 * ks][2], sc[2 * ks][3], pa[1]);
                pb[2] = pack2_rem(sc[2 * ks + 1][0], sc[2 * ks + 1][1], pa[2]);
                pb[3] = pack2_rem(sc[2 * ks + 1][2], sc[2 * ks + 1][3], pa[3]);
                l_run[0] += (sc[2 * ks][0] + sc[2 * ks][1]) + (sc[2 * ks + 1][0] + sc[2 * ks + 1][1]);
                l_run[1] += (sc[2 * ks][2] + sc[2 * ks][3]) + (sc[2 * ks + 1][2] + sc[2 * ks + 1][3]);
                const int vrow = ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                for (int n2 = 0; n2 < NT / 2; ++n2) {
                    uint32_t bfr[4];
                    ldmatrix_x4_trans(vbase + S::off(vrow, 2 * n2 + (lane >> 4)), bfr);
                    mma_bf16_16816(acc[2 * n2], pa, bfr[0], bfr[1]);
                    mma_bf16_16816(acc[2 * n2 + 1], pa, bfr[2], bfr[3]);
                    mma_bf16_16816(acc[2 * n2], pb, bfr[0], bfr[1]);
                    mma_bf16_16816(acc[2 * n2 + 1], pb, bfr[2], bfr[3]);
                }
            }
        }
        // normalise and store this tile's rows
#pragma unroll
        for (int h2 = 0; h2 < 2; ++h2) {
            float l = l_run[h2];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int t = row_t[h2];
            if (t < 0) continue;
            const float inv = 1.0f / l;
            uint32_t* orow = reinterpret_cast<uint32_t*>(O + ((size_t)b * k_h + row_kh[h2]) * Tlen * D + (size_t)t * D);
#pragma unroll
            for (int n = 0; n < NT; ++n)
                orow[n * 4 + tq] = pack2(acc[n][2 * h2] * inv, acc[n][2 * h2 + 1] * inv);
        }
    }
    // ---- context rows and zero rows, 16 bytes per store, in units of (head, 32 tokens) handed out
    // from a shared counter: the warps that had no row tile above take most of them
    const uint4* mean4 = reinterpret_cast<const uint4*>(s_mean);
    if (nwarps <= n_tiles) {
        // every warp had a row tile: they arrive together, a fixed split is cheaper than the counter
        for (int hh = 0; hh < rk; ++hh) {
            uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D);
            const uint32_t* bits = s_abits + hh * words;
            for (int i = threadIdx.x; i < Tlen * S::CPR; i += blockDim.x) {
                const int t = i / S::CPR, cc = i % S::CPR;
                if ((bits[t >> 5] >> (t & 31)) & 1u) continue;
                dst[i] = s_kind[t] ? mean4[cc] : make_uint4(0, 0, 0, 0);
            }
        }
        return;
    }
    const int blocks_per_head = (Tlen + 31) / 32;
    const int n_units = rk * blocks_per_head;
    for (;;) {
        int u = 0;
        if (lane == 0) u = atomicAdd(&s_fill_next, 1);
        u = __shfl_sync(0xffffffffu, u, 0);
        if (u >= n_units) break;
        const int hh = u / blocks_per_head, t0 = (u % blocks_per_head) * 32;
        uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D) + (size_t)t0 * S::CPR;
        const uint32_t abits = s_abits[hh * words + (t0 >> 5)];
#pragma unroll
        for (int i = lane; i < 32 * S::CPR; i += 32) {
            const int tl = i / S::CPR, cc = i % S::CPR;
            if (t0 + tl >= Tlen || ((abits >> tl) & 1u)) continue;
            dst[i] = s_kind[t0 + tl] ? mean4[cc] : make_uint4(0, 0, 0, 0);
        }
    }
}

template <int D>
size_t fused_smem_bytes(int T) {
    const int words = (T + 31) / 32;
    const int Tpad = (T + kKeyTile - 1) / kKeyTile * kKeyTile;
    size_t o = (((size_t)T * 2 + 127) / 128) * 128 + (((size_t)T + 127) / 128) * 128 +
               (((size_t)kMaxRK * words * 4 + 127) / 128) * 128 + (((size_t)kMaxRK * T * 4 + 127) / 128) * 128 +
               (size_t)kMaxRK * 256 * 4;
    return o + 2 * (size_t)Tpad * D * 2;
}

template <int D>
int launch_d(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    const sentry_attend_desc& d = a.d;
    const size_t fused_bytes = fused_smem_bytes<D>(d.T);
    if (fused_bytes <= 200 * 1024) {
        // the group's K and V fit in shared memory: one kernel does everything
        auto kern = attend_fused_bf16_kernel<D>;
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fused_bytes));
        // one big CTA, or two per SM; short sequences get small CTAs (more of them per SM: their
        // phases are a few barrier-separated microseconds each, so concurrency is what helps)
        const int threads = fused_bytes > 100 * 1024 ? 512 : (d.T <= kSmallT ? 128 : 256);
        LaunchScope ls(ctx, KS_ATT_CORE, st);
        kern<<<d.B * d.Hk, threads, fused_bytes, st>>>(
            (const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K, (const __nv_bfloat16*)a.V, a.kept_heads,
            a.ids, a.masks, a.sample_table, a.sample_offsets, a.n_subsets,
            a.selection_given ? a.active : nullptr, a.selection_given ? nullptr : a.active_out_user, d.T,
            d.Hq, d.Hk, d.k_h, d.c, d.score_mode, a.U_max, (__nv_bfloat16*)a.O, a.status, a.gate_scores, a.gate_S,
            a.kept_out);
        SENTRY_CUDA_TRY(cudaGetLastError());
        return SENTRY_OK;
    }
    if (a.gate_scores != nullptr) return SENTRY_ERR_UNSUPPORTED;   // the caller checks attend_bf16_gate_fusable
    const size_t valid_bytes = (((size_t)d.T * 2 + 127) / 128) * 128;
    // scores and selection by one CTA per group with K resident, where the shape allows it; the
    // streamed kernel then takes the active lists as given
    // (it needs about a CTA per SM to pay: with fewer groups than SMs the query-block score kernel,
    // which spreads a group over T/256 CTAs, is the faster one -- 0.32 against 0.52 ms on B=16, T=4096)
    const bool want_long = ctx->long_select == SENTRY_LONG_SELECT_PER_GROUP ||
                           (ctx->long_select == SENTRY_LONG_SELECT_AUTO && d.B * d.Hk >= ctx->sm_count);
    const bool long_select = !a.selection_given && want_long && attend_long_select_supported(d);
    if (long_select) {
        int rc = launch_attend_long_select(ctx, a, st);
        if (rc != SENTRY_OK) return rc;
    } else if (!a.selection_given) {
        // K segment: 64 KB worth of rows, a power of two (at most 8 segments for T <= 8192)
        int seg_shift = 0;
        while ((2 << seg_shift) * D * 2 <= 64 * 1024) ++seg_shift;
        while ((8 << seg_shift) < d.T) ++seg_shift;
        const int seg_rows = 1 << seg_shift;
        const size_t smem = valid_bytes + (size_t)kMaxActive * kScoreThreads * 2 + (size_t)seg_rows * D * 2;
        auto kern = attend_score_bf16_kernel<D>;
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        dim3 grid(d.B * d.Hk, (d.T + kScoreThreads - 1) / kScoreThreads);   // (sample, group) on x: no 65535 limit
        LaunchScope ls(ctx, KS_ATT_SCORE, st);
        kern<<<grid, kScoreThreads, smem, st>>>((const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K,
                                                 a.kept_heads, a.ids, a.masks, a.sample_table,
                                                 a.sample_offsets, a.n_subsets, d.T, d.Hq, d.Hk, d.k_h,
                                                 d.c, d.score_mode, seg_shift, a.mscore, a.status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    {
        const int words = (d.T + 31) / 32;
        size_t smem = valid_bytes + (((size_t)d.T + 127) / 128) * 128 +
                      (((size_t)kMaxRK * words * 4 + 127) / 128) * 128;
        size_t uni = CoreSmem<D>::PIPE_BYTES;
        const bool given = a.selection_given || long_select;
        if (!given && (size_t)kMaxRK * d.T * 4 > uni) uni = (size_t)kMaxRK * d.T * 4;
        smem += uni;
        auto kern = attend_core_bf16_kernel<D>;
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        LaunchScope ls(ctx, KS_ATT_CORE, st);
        kern<<<d.B * d.Hk, kCoreThreads, smem, st>>>(
            (const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K, (const __nv_bfloat16*)a.V, a.kept_heads,
            a.ids, a.masks, a.mscore, given ? a.active : nullptr,
            given ? nullptr : a.active_out_user, d.T, d.Hq, d.Hk, d.k_h, d.c, a.U_max,
            (__nv_bfloat16*)a.O, a.status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

}  // namespace

// bf16, at most 4 query heads per KV group, U <= 48 and shared memory within reach.
bool attend_bf16_supported(const sentry_attend_desc& d) {
    if (d.dtype != ATT_DTYPE) return false;
    if (d.Hq / d.Hk > kMaxRK) return false;
    if (sentry_num_active(d.T, d.c) > kMaxActive) return false;
    if (d.T > 8192) return false;
    return d.d == 16 || d.d == 32 || d.d == 64;
}

// Whether the head selection can ride inside the attention launch: the fused kernel (K and V of a
// group resident in shared memory) with at most 64 heads.
bool attend_bf16_gate_fusable(const sentry_attend_desc& d) {
    if (!attend_bf16_supported(d) || d.Hq > 64 || d.k_h > 64) return false;
    switch (d.d) {
        case 16: return fused_smem_bytes<16>(d.T) <= 200 * 1024;
        case 32: return fused_smem_bytes<32>(d.T) <= 200 * 1024;
        case 64: return fused_smem_bytes<64>(d.T) <= 200 * 1024;
        default: return false;
    }
}

int launch_attend_bf16(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    switch (a.d.d) {
        case 16: return launch_d<16>(ctx, a, st);
        case 32: return launch_d<32>(ctx, a, st);
        case 64: return launch_d<64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

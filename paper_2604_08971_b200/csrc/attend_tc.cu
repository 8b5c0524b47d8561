// SentryAttend (Section 4.4, Eq. 6) for bf16 tensors on the 5th-generation tensor cores, for
// sequences whose K and V rows of one KV group fit in shared memory (T up to ~1.3 k at d = 32).
//
// One CTA per (sample, KV group) does everything for the group's kept heads:
//   1. present tokens of the sample -> runs of consecutive tokens.  Every run is brought in by
//      TMA tensor copies (boxes of 64 and of 8 rows, no multicast) into the swizzled row layout
//      the tensor core reads; the last len % 8 rows of a run, and everything when the present
//      tokens are scattered over more than kMaxRuns runs, come by 16-byte async copies into the
//      same layout.  Run starts sit on 8-row boundaries; the rows in between are zero and are
//      masked out of every softmax.  K and V are read from HBM once per group.
//   2. sparsity score of every present query on its sampled keys, all kept heads of the group
//      in one pass over the resident K rows (fp32 accumulation of exact bf16 products).
//   3. top-U selection per head (ties -> lower index).
//   4. Eq. 6 on the active rows: the U rows of all kept heads of the group are stacked into
//      M = 128 row tiles; per 64-key tile  S = Q_act K^T  (tcgen05.mma, fp32 in TMEM), softmax
//      weights by four warps that own one accumulator row per lane (pass 1: row maxima,
//      pass 2: p = 2^((s - max) c), bf16, written to shared memory as the next A operand),
//      O += P V  with V read in place as an MN-major operand, and the normaliser
//      l += P 1  from the same rounded weights on the tensor core.
//   5. meanwhile the other warps sum the columns of V (the context vector) and write the context
//      rows and the zero rows of absent tokens; the softmax warps finish with O / l on their rows.
// Every wait is bounded; on expiry the CTA raises SENTRY_STATUS_BIT_TIMEOUT and unwinds.
#include <cuda.h>

#include "attend_common.cuh"
#include "tc_common.cuh"

namespace {

constexpr int kMaxRuns = 16;       // runs of consecutive present tokens fetched by TMA
constexpr int kKT = 64;            // keys per S tile
constexpr int kTmemColsAtt = 256;  // S0 | S1 | O | l
constexpr int kColS0 = 0, kColS1 = 64, kColO = 128, kColL = 192;
constexpr int kPBytes = 128 * 128;  // one P tile: 128 rows x 64 keys bf16, 128-byte rows
constexpr int kIssuerWarp = 0, kSoftmaxWarp0 = 4;

struct AttMisc {
    uint64_t k_full, v_full;
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full[2], p_empty[2];
    uint64_t o_full, o_empty;
    uint32_t tmem_base;
    int abort_flag;
    int n_runs, t_pad;
    int run_p[kMaxRuns + 1];     // first compact position of each run (+ end)
    int run_row[kMaxRuns];       // first shared-memory row of each run (multiple of 8)
    int pick[2];
    int cls[33];
    int wcnt[32];
};

// bytes of dynamic shared memory; the kernel carves it in the same order
template <int D>
struct AttSmem {
    static constexpr int RB = D * 2;
    int rows_cap, nmt, T;
    size_t off_v, off_q, off_p, off_ones, off_misc, off_valid, off_prow, off_kind, off_abits, off_kbits,
        off_keys, off_hist, total;
    __host__ __device__ AttSmem(int T_, int nmt_) : T(T_) {
        const int max_runs = T_ / 2 + 1 < kMaxRuns ? T_ / 2 + 1 : kMaxRuns;
        rows_cap = (T_ + 7 * (max_runs - 1) + kKT - 1) / kKT * kKT;
        nmt = nmt_;
        size_t o = 0;
        o += (size_t)rows_cap * RB;  o = (o + 1023) / 1024 * 1024;  off_v = o;
        o += (size_t)rows_cap * RB;  o = (o + 1023) / 1024 * 1024;  off_q = o;
        o += (size_t)nmt * 128 * RB; o = (o + 1023) / 1024 * 1024;  off_p = o;
        o += 2 * (size_t)kPBytes;                                    off_ones = o;
        o += 512;                                                    off_misc = o;
        o += (sizeof(AttMisc) + 127) / 128 * 128;                    off_valid = o;
        o += ((size_t)T_ * 2 + 127) / 128 * 128;                     off_prow = o;
        o += ((size_t)T_ * 2 + 127) / 128 * 128;                     off_kind = o;
        o += ((size_t)T_ + 127) / 128 * 128;                         off_abits = o;
        o += ((size_t)kMaxRK * ((T_ + 31) / 32) * 4 + 127) / 128 * 128;  off_kbits = o;
        o += ((size_t)(rows_cap / 32) * 4 + 127) / 128 * 128;        off_keys = o;
        o += ((size_t)kMaxRK * T_ * 4 + 127) / 128 * 128;            off_hist = o;
        o += (size_t)kMaxRK * 256 * 4;
        total = o + 1024;   // alignment slack
    }
};

__device__ __forceinline__ void bar_sync_group(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void tmem_ld_32x1(uint32_t taddr, uint32_t& r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r) : "r"(taddr) : "memory");
}

// Sparsity scores (Section 4.4) of NH heads of the group at once for the queries of this thread:
// M_i = max_j s_ij - mean_j s_ij over the sampled (or all) present keys, s_ij = q_i.k_j / sqrt(d),
// K rows from shared memory.  The query rows stay in registers as packed bf16, so a sampled key row
// is fetched once per group.  The 1/sqrt(d) factor is applied once at the end (it is positive, so it
// commutes with the maximum).  PAD: compact key positions map to rows through prow (runs start on
// 8-row boundaries); otherwise position = row.
template <int D, int NH, bool PAD>
__device__ __forceinline__ void score_pass_tc(const __nv_bfloat16* __restrict__ Q, const size_t* q_base,
                                              const uint16_t* s_valid, const uint16_t* s_prow, uint32_t ks_addr,
                                              int Tv, const int32_t* __restrict__ tbl, int n_s, int cnt,
                                              int score_mode, uint32_t* const* keys_out, unsigned int* status) {
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
        const int32_t* row = score_mode == 0 ? tbl + (size_t)p * n_s : nullptr;
        int pj_next = score_mode == 0 ? __ldg(row) : 0;
        for (int a = 0; a < cnt; ++a) {
            int pj = pj_next;
            if (a + 1 < cnt) pj_next = score_mode == 0 ? __ldg(row + a + 1) : a + 1;
            if (pj < 0 || pj >= Tv) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); pj = 0; }
            const int r = PAD ? (int)s_prow[pj] : pj;
            float acc[NH][4];
#pragma unroll
            for (int h = 0; h < NH; ++h) acc[h][0] = acc[h][1] = acc[h][2] = acc[h][3] = 0.f;
#pragma unroll
            for (int cc = 0; cc < S::CPR; ++cc) {
                const uint4 v = lds128(ks_addr + S::off(r, cc));
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
                const float sc = (acc[h][0] + acc[h][1]) + (acc[h][2] + acc[h][3]);
                mx[h] = fmaxf(mx[h], sc);
                sum[h] += sc;
            }
        }
#pragma unroll
        for (int h = 0; h < NH; ++h) keys_out[h][p] = sentry_order_key((mx[h] - sum[h] * inv_cnt) * scale);
    }
}

template <int D, bool PAD>
__device__ __forceinline__ void score_heads_tc(const __nv_bfloat16* __restrict__ Q, int b, int Hq, int Tlen, int rk,
                                               const int* hs, const uint16_t* s_valid, const uint16_t* s_prow,
                                               uint32_t ks_addr, int Tv, const int32_t* tbl, int n_s, int cnt,
                                               int score_mode, uint32_t* s_keys, unsigned int* status) {
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
#define SCORE_PASS(N) score_pass_tc<D, N, PAD>(Q, q_base, s_valid, s_prow, ks_addr, Tv, tbl, n_s, cnt, score_mode, \
                                               keys_out, status)
        if (nh == 1) SCORE_PASS(1);
        else if (nh == 2) SCORE_PASS(2);
        else if constexpr (HPP == 4) {
            if (nh == 3) SCORE_PASS(3);
            else SCORE_PASS(4);
        }
#undef SCORE_PASS
    }
}

// grid B*Hk; 256 or 512 threads.  tm_*64 / tm_*8: maps over K and V viewed as [B*Hk*T, D] with
// boxes of 64 and 8 rows.
template <int D>
__global__ void __launch_bounds__(512, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap tm_k64, const __grid_constant__ CUtensorMap tm_k8,
                 const __grid_constant__ CUtensorMap tm_v64, const __grid_constant__ CUtensorMap tm_v8,
                 const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                 const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ kept_heads,
                 const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks,
                 const int32_t* __restrict__ table, const int64_t* __restrict__ offsets, int n_subsets,
                 const int32_t* __restrict__ active_in, int32_t* __restrict__ active_out, int Tlen, int Hq,
                 int Hk, int k_h, int c, int score_mode, int U_max, int nmt_cap,
                 __nv_bfloat16* __restrict__ O, unsigned int* status) {
    using S = Sw<D>;
    constexpr int RB = D * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ int red[66];
    __shared__ int32_t s_act[kMaxRK][kMaxActive];
    __shared__ float s_vpart[512 / (D / 2)][D];
    __shared__ __align__(16) __nv_bfloat16 s_mean[D];

    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    const AttSmem<D> L(Tlen, nmt_cap);
    const uint32_t ks_addr = base, vs_addr = base + (uint32_t)L.off_v, qs_addr = base + (uint32_t)L.off_q,
                   ps_addr = base + (uint32_t)L.off_p, ones_addr = base + (uint32_t)L.off_ones;
    AttMisc* misc = reinterpret_cast<AttMisc*>(smem + L.off_misc);
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(smem + L.off_valid);
    uint16_t* s_prow = reinterpret_cast<uint16_t*>(smem + L.off_prow);
    uint8_t* s_kind = smem + L.off_kind;
    uint32_t* s_abits = reinterpret_cast<uint32_t*>(smem + L.off_abits);
    uint32_t* s_kbits = reinterpret_cast<uint32_t*>(smem + L.off_kbits);
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem + L.off_keys);
    int* s_hist = reinterpret_cast<int*>(smem + L.off_hist);
    volatile int* abort_flag = &misc->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int words = (Tlen + 31) / 32;

    // Samples with more modalities present take longer; in small batches the CTAs take them
    // heaviest first (every CTA finds the sample of its rank by itself with a counting sort on
    // the number of present modalities), so that the long ones do not end up alone in the tail
    // of the launch.
    int b = blockIdx.x / Hk;
    const int g = blockIdx.x % Hk;
    const int Bn = gridDim.x / Hk;
    if (Bn > 1 && Bn <= kOrderMaxBatch) {
        if (threadIdx.x < 33) misc->cls[threadIdx.x] = 0;
        __syncthreads();
        for (int bb = threadIdx.x; bb < Bn; bb += blockDim.x) atomicAdd(&misc->cls[__popc(masks[bb])], 1);
        __syncthreads();
        if (threadIdx.x == 0) {   // class (present modalities, descending) that holds rank b, and the offset in it
            int left = b, cls = 32;
            while (cls > 0 && left >= misc->cls[cls]) { left -= misc->cls[cls]; --cls; }
            misc->pick[0] = cls;
            misc->pick[1] = left;
        }
        __syncthreads();
        const int cls = misc->pick[0];
        int need = misc->pick[1];      // the need-th sample of that class, in index order
        __syncthreads();
        for (int b0 = 0; b0 < Bn; b0 += blockDim.x) {
            const int bb = b0 + threadIdx.x;
            const bool hit = bb < Bn && __popc(masks[bb]) == cls;
            const unsigned bm = __ballot_sync(0xffffffffu, hit);
            if (lane == 0) misc->wcnt[warp] = __popc(bm);
            __syncthreads();
            int before = 0, tot = 0;
            for (int w = 0; w < nwarps; ++w) { if (w < warp) before += misc->wcnt[w]; tot += misc->wcnt[w]; }
            if (hit && before + __popc(bm & ((1u << lane) - 1u)) == need) misc->pick[0] = bb;
            __syncthreads();
            if (need < tot) break;
            need -= tot;
        }
        __syncthreads();
        b = misc->pick[0];
    }
    const uint32_t mask = masks[b];
    const int Tv = block_build_valid(ids, Tlen, mask, s_valid, red);
    int hs[kMaxRK], khs[kMaxRK];
    bool bad;
    const int rk = group_heads(kept_heads + (size_t)b * k_h, k_h, Hq / Hk, g, Hq, hs, khs, bad);
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

    // ---- barriers, tensor memory, runs of consecutive present tokens
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&misc->k_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->v_full), 1);
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&misc->s_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&misc->s_empty[i]), 4);
            ptx::mbar_init(ptx::smem_u32(&misc->p_full[i]), 4);
            ptx::mbar_init(ptx::smem_u32(&misc->p_empty[i]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&misc->o_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->o_empty), 4);
        misc->abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), kTmemColsAtt);
        ptx::tmem_relinquish();
        // run starts: positions whose token does not follow the previous present token
        int nr = 0;
        for (int p0 = 0; p0 < Tv; p0 += 32) {
            const int p = p0 + lane;
            const bool start = p < Tv && (p == 0 || s_valid[p] != s_valid[p - 1] + 1);
            const unsigned bm = __ballot_sync(0xffffffffu, start);
            if (start) {
                const int idx = nr + __popc(bm & ((1u << lane) - 1u));
                if (idx < kMaxRuns) misc->run_p[idx] = p;
            }
            nr += __popc(bm);
        }
        __syncwarp();
        if (lane == 0) {
            if (nr > kMaxRuns) {        // scattered tokens: one unpadded list, fetched row by row
                misc->n_runs = 0;
                misc->t_pad = Tv;
            } else {
                misc->run_p[nr] = Tv;
                int row = 0;
                for (int k = 0; k < nr; ++k) {
                    misc->run_row[k] = row;
                    row += misc->run_p[k + 1] - misc->run_p[k];
                    if (k + 1 < nr) row = (row + 7) & ~7;
                }
                misc->n_runs = nr;
                misc->t_pad = row;
            }
        }
    }
    for (int i = threadIdx.x; i < L.rows_cap / 32; i += blockDim.x) s_kbits[i] = 0u;
    for (int t = threadIdx.x; t < Tlen; t += blockDim.x) s_kind[t] = 0;
    for (int i = threadIdx.x; i < kMaxRK * words; i += blockDim.x) s_abits[i] = 0u;
    for (int i = threadIdx.x; i < kMaxRK * kMaxActive; i += blockDim.x) (&s_act[0][0])[i] = -1;
    if (threadIdx.x < 128) reinterpret_cast<uint32_t*>(smem + L.off_ones)[threadIdx.x] = 0x3f803f80u;  // bf16 1.0
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = misc->tmem_base;
    const int n_runs = misc->n_runs;
    const int Tp = misc->t_pad;
    const bool padded = Tp != Tv;
    const int n_kt = (Tp + kKT - 1) / kKT;
    const int rows_staged = n_kt * kKT;
    const __nv_bfloat16* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    const __nv_bfloat16* Vg = V + ((size_t)b * Hk + g) * Tlen * D;

    // ---- stage K, then V: TMA boxes for whole groups of 8 rows of every run
    if (warp == 0) {
        if (elect_one()) {
            uint32_t bytes = 0;
            for (int k = 0; k < n_runs; ++k) bytes += (uint32_t)((misc->run_p[k + 1] - misc->run_p[k]) & ~7) * RB;
            const int grow0 = (b * Hk + g) * Tlen;
            for (int which = 0; which < 2; ++which) {
                const uint32_t bar = ptx::smem_u32(which == 0 ? &misc->k_full : &misc->v_full);
                const uint32_t dst0 = which == 0 ? ks_addr : vs_addr;
                const CUtensorMap* m64 = which == 0 ? &tm_k64 : &tm_v64;
                const CUtensorMap* m8 = which == 0 ? &tm_k8 : &tm_v8;
                ptx::mbar_arrive_expect_tx(bar, bytes);
                for (int k = 0; k < n_runs; ++k) {
                    const int p0 = misc->run_p[k], len = misc->run_p[k + 1] - p0;
                    const int y0 = grow0 + (int)s_valid[p0];
                    const uint32_t dst = dst0 + (uint32_t)misc->run_row[k] * RB;
                    int o = 0;
                    for (; o + 64 <= len; o += 64) ptx::tma_load_2d(dst + o * RB, m64, 0, y0 + o, bar);
                    for (; o + 8 <= len; o += 8) ptx::tma_load_2d(dst + o * RB, m8, 0, y0 + o, bar);
                }
            }
        }
        __syncwarp();
    }
    // compact position -> row, key-validity bits
    if (n_runs == 0) {
        for (int p = threadIdx.x; p < Tv; p += blockDim.x) s_prow[p] = (uint16_t)p;
    } else {
        for (int k = 0; k < n_runs; ++k) {
            const int p0 = misc->run_p[k], len = misc->run_p[k + 1] - p0, r0 = misc->run_row[k];
            for (int o = threadIdx.x; o < len; o += blockDim.x) s_prow[p0 + o] = (uint16_t)(r0 + o);
        }
    }
    __syncthreads();
    for (int p = threadIdx.x; p < Tv; p += blockDim.x) {
        const int r = s_prow[p];
        atomicOr(&s_kbits[r >> 5], 1u << (r & 31));
        s_kind[s_valid[p]] = 1;
    }
    // rows that TMA does not bring: run tails (len % 8 rows), or every row of a scattered list
    if (n_runs == 0) {
        for (int i = threadIdx.x; i < Tv * S::CPR; i += blockDim.x) {
            const int p = i / S::CPR, cc = i % S::CPR;
            const size_t goff = (size_t)s_valid[p] * D + cc * 8;
            ptx::cp_async_16(ks_addr + S::off(p, cc), Kg + goff);
            ptx::cp_async_16(vs_addr + S::off(p, cc), Vg + goff);
        }
    } else {
        for (int i = threadIdx.x; i < n_runs * 7 * S::CPR; i += blockDim.x) {
            const int k = i / (7 * S::CPR), o7 = (i / S::CPR) % 7, cc = i % S::CPR;
            const int p0 = misc->run_p[k], len = misc->run_p[k + 1] - p0;
            if (o7 < (len & 7)) {
                const int p = p0 + (len & ~7) + o7;
                const int r = misc->run_row[k] + (len & ~7) + o7;
                const size_t goff = (size_t)s_valid[p] * D + cc * 8;
                ptx::cp_async_16(ks_addr + S::off(r, cc), Kg + goff);
                ptx::cp_async_16(vs_addr + S::off(r, cc), Vg + goff);
            }
        }
    }
    ptx::cp_async_commit();
    __syncthreads();   // s_kbits complete
    // zero the rows between runs and behind the last one (they are masked, but must be finite)
    for (int i = threadIdx.x; i < rows_staged * S::CPR; i += blockDim.x) {
        const int r = i / S::CPR, cc = i % S::CPR;
        if (!((s_kbits[r >> 5] >> (r & 31)) & 1u)) {
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(ks_addr + S::off(r, cc)), "r"(0) : "memory");
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vs_addr + S::off(r, cc)), "r"(0) : "memory");
        }
    }
    ptx::cp_async_wait_all();
    bool ok = __syncthreads_and(warp_wait(&misc->k_full, 0u, abort_flag) ? 1 : 0) != 0;   // block-uniform

    if (ok && active_in == nullptr) {
        // ---- sparsity scores (Section 4.4) from the resident K rows
        const int n_s = U;
        const int cnt = score_mode == 0 ? n_s : Tv;
        const int32_t* tbl = nullptr;
        bool table_ok = true;
        if (score_mode == 0) {
            if (mask >= (uint32_t)n_subsets || offsets[mask] < 0) table_ok = false;
            else tbl = table + offsets[mask];
        }
        if (table_ok) {
            if (padded) score_heads_tc<D, true>(Q, b, Hq, Tlen, rk, hs, s_valid, s_prow, ks_addr, Tv, tbl, n_s, cnt,
                                                score_mode, s_keys, status);
            else score_heads_tc<D, false>(Q, b, Hq, Tlen, rk, hs, s_valid, s_prow, ks_addr, Tv, tbl, n_s, cnt,
                                          score_mode, s_keys, status);
        } else {
            if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            for (int i = threadIdx.x; i < rk * Tlen; i += blockDim.x) s_keys[i] = 0u;
        }
        __syncthreads();
        // ---- the U present queries with the largest score are active
        if (Tv <= 256) warps_select_topk_heads(s_keys, Tlen, Tv, U, rk, s_act, s_valid);
        else block_select_topk_heads(s_keys, Tlen, Tv, U, rk, s_act, s_valid, s_hist);
        __syncthreads();
        if (active_out != nullptr)
            for (int i = threadIdx.x; i < rk * U_max; i += blockDim.x) {
                const int hh = i / U_max, a = i % U_max;
                active_out[((size_t)b * k_h + khs[hh]) * U_max + a] = a < U ? s_act[hh][a] : -1;
            }
    } else if (ok) {
        for (int i = threadIdx.x; i < rk * kMaxActive; i += blockDim.x) {
            const int hh = i / kMaxActive, a = i % kMaxActive;
            int t = a < U_max ? active_in[((size_t)b * k_h + khs[hh]) * U_max + a] : -1;
            if (t >= 0 && (t >= Tlen || s_kind[t] == 0)) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); t = -1; }
            s_act[hh][a] = t;
        }
        __syncthreads();
    }

    // ---- stacked active rows: row m = hh * UA + a  <->  (kept head hh of the group, a-th active token)
    const int UA = min(U, kMaxActive);
    const int R = rk * UA;
    const int nmt = (R + 127) / 128;
    if (ok) {
        for (int i = threadIdx.x; i < rk * kMaxActive; i += blockDim.x) {
            const int hh = i / kMaxActive, t = s_act[hh][i % kMaxActive];
            if (t >= 0) atomicOr(&s_abits[hh * words + (t >> 5)], 1u << (t & 31));
        }
        for (int i = threadIdx.x; i < nmt * 128 * S::CPR; i += blockDim.x) {
            const int m = i / S::CPR, cc = i % S::CPR;
            const int hh = m / UA, a = m - hh * UA;
            const int t = m < R ? s_act[hh][a] : -1;
            const uint32_t dst = qs_addr + S::off(m, cc);
            if (t >= 0) ptx::cp_async_16(dst, Q + ((size_t)b * Hq + hs[hh]) * Tlen * D + (size_t)t * D + cc * 8);
            else asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
        }
        ptx::cp_async_wait_all();
        ok = warp_wait(&misc->v_full, 0u, abort_flag);
    }
    ptx::fence_proxy_async_smem();   // zero rows, tail rows and gathered Q rows -> visible to the tensor core
    ok = __syncthreads_and(ok ? 1 : 0) != 0;

    const uint32_t mb = ptx::smem_u32(misc);
    auto BAR = [&](size_t off) { return mb + (uint32_t)off; };
    if (!ok) {
        // fall through to the teardown
    } else if (warp == kIssuerWarp) {
        // ------------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc_qk = ptx::umma_idesc_bf16(128, kKT);
        constexpr uint32_t idesc_pv = ptx::umma_idesc_bf16_major(128, D, false, true);
        constexpr uint32_t idesc_l = ptx::umma_idesc_bf16_major(128, 16, false, true);
        const uint64_t ones_desc = ptx::umma_smem_desc_rows(ones_addr, 32);
        uint32_t n = 0, m = 0;
        bool iok = true;
        auto issue_qk = [&](int mt, int t) {
            const uint32_t buf = n & 1u;
            iok = warp_wait(&misc->s_empty[buf], ((n >> 1) & 1u) ^ 1u, abort_flag);
            if (!iok) return;
            ptx::tc_fence_after_sync();
            if (elect_one()) {
                const uint32_t d_tm = tmem + (buf ? kColS1 : kColS0);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint64_t a = ptx::umma_smem_desc_rows(qs_addr + (uint32_t)mt * 128 * RB + ks * 32, RB);
                    const uint64_t bd = ptx::umma_smem_desc_rows(ks_addr + (uint32_t)t * kKT * RB + ks * 32, RB);
                    ptx::umma_bf16(d_tm, a, bd, idesc_qk, ks > 0 ? 1u : 0u);
                }
                ptx::umma_commit(ptx::smem_u32(&misc->s_full[buf]));
            }
            __syncwarp();
            ++n;
        };
        auto issue_pv = [&](int mt, int t, bool last) {
            const uint32_t buf = m & 1u;
            if (t == 0) iok = warp_wait(&misc->o_empty, ((uint32_t)mt & 1u) ^ 1u, abort_flag);
            if (iok) iok = warp_wait(&misc->p_full[buf], (m >> 1) & 1u, abort_flag);
            if (!iok) return;
            ptx::tc_fence_after_sync();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kKT / 16; ++kk) {
                    const uint64_t a = ptx::umma_smem_desc_sw128(ps_addr + buf * kPBytes + kk * 32);
                    const uint64_t bd = ptx::umma_smem_desc_rows(vs_addr + (uint32_t)(t * kKT + kk * 16) * RB, RB);
                    const uint32_t acc = (t > 0 || kk > 0) ? 1u : 0u;
                    ptx::umma_bf16(tmem + kColO, a, bd, idesc_pv, acc);
                    ptx::umma_bf16(tmem + kColL, a, ones_desc, idesc_l, acc);
                }
                ptx::umma_commit(ptx::smem_u32(&misc->p_empty[buf]));
                if (last) ptx::umma_commit(ptx::smem_u32(&misc->o_full));
            }
            __syncwarp();
            ++m;
        };
        for (int mt = 0; mt < nmt && iok; ++mt) {
            for (int t = 0; t < n_kt && iok; ++t) issue_qk(mt, t);             // pass 1: row maxima
            for (int t = 0; t < n_kt && iok; ++t) {                            // pass 2: weights, P V
                issue_qk(mt, t);
                if (t > 0 && iok) issue_pv(mt, t - 1, false);
            }
            if (iok) issue_pv(mt, n_kt - 1, true);
        }
    } else if (warp >= kSoftmaxWarp0 && warp < kSoftmaxWarp0 + 4) {
        // ----------------------------------------------------------------- softmax warps
        const int quarter = warp & 3;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const float cl2 = rsqrtf((float)D) * 1.4426950408889634f;   // 1/sqrt(d) * log2(e)
        uint32_t n = 0, m = 0;
        bool sok = true;
        for (int mt = 0; mt < nmt && sok; ++mt) {
            const int row = mt * 128 + quarter * 32 + lane;
            const bool warp_has_rows = mt * 128 + quarter * 32 < R;
            float mx = -INFINITY;
            for (int pass = 0; pass < 2 && sok; ++pass) {
                const float shift = -mx * cl2;   // pass 2
                for (int t = 0; t < n_kt && sok; ++t) {
                    const uint32_t buf = n & 1u;
                    sok = warp_wait(&misc->s_full[buf], (n >> 1) & 1u, abort_flag);
                    if (!sok) break;
                    ++n;
                    ptx::tc_fence_after_sync();
                    uint32_t s0[32], s1[32];
                    const uint32_t tcol = lane_base + (buf ? kColS1 : kColS0);
                    if (warp_has_rows) {
                        ptx::tmem_ld_32x32(tcol, s0);
                        ptx::tmem_ld_32x32(tcol + 32, s1);
                        ptx::tmem_ld_wait();
                    }
                    ptx::tc_fence_before_sync();
                    warp_arrive(&misc->s_empty[buf]);
                    const uint32_t kb0 = s_kbits[2 * t], kb1 = s_kbits[2 * t + 1];
                    if (pass == 0) {
                        if (!warp_has_rows) continue;
                        if ((kb0 & kb1) == 0xffffffffu) {
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                mx = max3(mx, __uint_as_float(s0[i]), __uint_as_float(s0[i + 1]));
                                mx = max3(mx, __uint_as_float(s1[i]), __uint_as_float(s1[i + 1]));
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                if ((kb0 >> i) & 1u) mx = fmaxf(mx, __uint_as_float(s0[i]));
                                if ((kb1 >> i) & 1u) mx = fmaxf(mx, __uint_as_float(s1[i]));
                            }
                        }
                        continue;
                    }
                    // pass 2: weights of this tile -> bf16 -> shared memory (A operand of P V)
                    uint32_t pk[32];
                    if (warp_has_rows) {
                        if ((kb0 & kb1) == 0xffffffffu) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                pk[i] = pack2(fast_exp2(fmaf(__uint_as_float(s0[2 * i]), cl2, shift)),
                                              fast_exp2(fmaf(__uint_as_float(s0[2 * i + 1]), cl2, shift)));
                                pk[16 + i] = pack2(fast_exp2(fmaf(__uint_as_float(s1[2 * i]), cl2, shift)),
                                                   fast_exp2(fmaf(__uint_as_float(s1[2 * i + 1]), cl2, shift)));
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const float a0 = ((kb0 >> (2 * i)) & 1u) ? fast_exp2(fmaf(__uint_as_float(s0[2 * i]), cl2, shift)) : 0.f;
                                const float a1 = ((kb0 >> (2 * i + 1)) & 1u) ? fast_exp2(fmaf(__uint_as_float(s0[2 * i + 1]), cl2, shift)) : 0.f;
                                const float b0 = ((kb1 >> (2 * i)) & 1u) ? fast_exp2(fmaf(__uint_as_float(s1[2 * i]), cl2, shift)) : 0.f;
                                const float b1 = ((kb1 >> (2 * i + 1)) & 1u) ? fast_exp2(fmaf(__uint_as_float(s1[2 * i + 1]), cl2, shift)) : 0.f;
                                pk[i] = pack2(a0, a1);
                                pk[16 + i] = pack2(b0, b1);
                            }
                        }
                    }
                    const uint32_t pbuf = m & 1u;
                    sok = warp_wait(&misc->p_empty[pbuf], ((m >> 1) & 1u) ^ 1u, abort_flag);
                    if (!sok) break;
                    ++m;
                    if (warp_has_rows) {
                        const int prow = quarter * 32 + lane;
                        const uint32_t dst_row = ps_addr + pbuf * kPBytes + prow * 128;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst_row + ((i ^ (prow & 7)) << 4)),
                                         "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]), "r"(pk[4 * i + 3])
                                         : "memory");
                        }
                    }
                    ptx::fence_proxy_async_smem();
                    warp_arrive(&misc->p_full[pbuf]);
                }
            }
            if (!sok) break;
            // ---- rows of this tile: O / l -> bf16 -> global
            sok = warp_wait(&misc->o_full, (uint32_t)mt & 1u, abort_flag);
            if (!sok) break;
            ptx::tc_fence_after_sync();
            uint32_t o[D], lw = 0;
            if (warp_has_rows) {
                if constexpr (D == 16) {
                    ptx::tmem_ld_32x16(lane_base + kColO, reinterpret_cast<uint32_t(&)[16]>(o));
                } else {
#pragma unroll
                    for (int j = 0; j < D / 32; ++j)
                        ptx::tmem_ld_32x32(lane_base + kColO + 32 * j, reinterpret_cast<uint32_t(&)[32]>(o[32 * j]));
                }
                tmem_ld_32x1(lane_base + kColL, lw);
                ptx::tmem_ld_wait();
            }
            ptx::tc_fence_before_sync();
            warp_arrive(&misc->o_empty);
            if (warp_has_rows && row < R) {
                const int hh = row / UA, a = row - hh * UA;
                const int tkn = s_act[hh][a];
                if (tkn >= 0) {
                    const float inv = 1.0f / __uint_as_float(lw);
                    uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D + (size_t)tkn * D);
#pragma unroll
                    for (int cc = 0; cc < D / 8; ++cc) {
                        uint4 v;
                        v.x = pack2(__uint_as_float(o[8 * cc]) * inv, __uint_as_float(o[8 * cc + 1]) * inv);
                        v.y = pack2(__uint_as_float(o[8 * cc + 2]) * inv, __uint_as_float(o[8 * cc + 3]) * inv);
                        v.z = pack2(__uint_as_float(o[8 * cc + 4]) * inv, __uint_as_float(o[8 * cc + 5]) * inv);
                        v.w = pack2(__uint_as_float(o[8 * cc + 6]) * inv, __uint_as_float(o[8 * cc + 7]) * inv);
                        dst[cc] = v;
                    }
                }
            }
        }
    } else {
        // ------------------------------------------- context vector, context rows and zero rows
        // fill group: every warp except the issuer and the softmax warps
        const int n_fill = (int)blockDim.x - 5 * 32;
        const int ft = warp < kSoftmaxWarp0 ? (int)threadIdx.x - 32 : (int)threadIdx.x - 5 * 32;
        constexpr int DP = D / 2;
        const int vs_dp = ft % DP, vs_k0 = ft / DP;
        const int stride = n_fill / DP;
        float v0 = 0.f, v1 = 0.f;
        if (vs_k0 < stride) {
            for (int r = vs_k0; r < rows_staged; r += stride) {   // padding rows are zero
                uint32_t w;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(vs_addr + S::off(r, vs_dp >> 2) + (vs_dp & 3) * 4));
                v0 += __uint_as_float(w << 16);
                v1 += __uint_as_float(w & 0xffff0000u);
            }
            s_vpart[vs_k0][2 * vs_dp] = v0;
            s_vpart[vs_k0][2 * vs_dp + 1] = v1;
        }
        bar_sync_group(1, n_fill);
        if (ft < D) {
            float t = 0.f;
            for (int i = 0; i < stride; ++i) t += s_vpart[i][ft];
            s_mean[ft] = __float2bfloat16_rn(t / (float)Tv);
        }
        bar_sync_group(1, n_fill);
        const uint4* mean4 = reinterpret_cast<const uint4*>(s_mean);
        for (int hh = 0; hh < rk; ++hh) {
            uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D);
            const uint32_t* bits = s_abits + hh * words;
            for (int i = ft; i < Tlen * S::CPR; i += n_fill) {
                const int t = i / S::CPR, cc = i % S::CPR;
                if ((bits[t >> 5] >> (t & 31)) & 1u) continue;
                dst[i] = s_kind[t] ? mean4[cc] : make_uint4(0, 0, 0, 0);
            }
        }
    }

    // ---------------------------------------------------------------------------- teardown
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
        ptx::tmem_dealloc(tmem, kTmemColsAtt);
    }
}

template <int D>
int launch_d(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    const sentry_attend_desc& d = a.d;
    const int r = d.Hq / d.Hk;
    const int ua = a.U_max < kMaxActive ? a.U_max : kMaxActive;
    const int nmt = ((r < kMaxRK ? r : kMaxRK) * ua + 127) / 128;
    const AttSmem<D> L(d.T, nmt);
    const uint64_t rows = (uint64_t)d.B * d.Hk * d.T;
    CUtensorMap k64, k8, v64, v8;
    if (!make_map_2d(&k64, a.K, rows, D, 64, D) || !make_map_2d(&k8, a.K, rows, D, 8, D) ||
        !make_map_2d(&v64, a.V, rows, D, 64, D) || !make_map_2d(&v8, a.V, rows, D, 8, D))
        return SENTRY_ERR_CUDA;
    auto kern = attend_tc_kernel<D>;
    // two CTAs per SM at most (each holds 256 of the 512 tensor-memory columns)
    size_t smem = L.total;
    if (smem < 80 * 1024) smem = 80 * 1024;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int threads = smem > 110 * 1024 ? 512 : 256;
    LaunchScope ls(ctx, KS_ATT_CORE, st);
    kern<<<d.B * d.Hk, threads, smem, st>>>(
        k64, k8, v64, v8, (const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K, (const __nv_bfloat16*)a.V,
        a.kept_heads, a.ids, a.masks, a.sample_table, a.sample_offsets, a.n_subsets,
        a.selection_given ? a.active : nullptr, a.selection_given ? nullptr : a.active_out_user, d.T, d.Hq, d.Hk,
        d.k_h, d.c, d.score_mode, a.U_max, nmt, (__nv_bfloat16*)a.O, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

}  // namespace

// bf16, at most kMaxRK query heads per KV group, U <= kMaxActive, and K, V of a group (plus the
// working buffers) within the shared memory of one SM.
bool attend_tc_supported(const sentry_attend_desc& d) {
    if (d.dtype != SENTRY_BF16) return false;
    if (d.Hq / d.Hk > kMaxRK) return false;
    const int U_max = sentry_num_active(d.T, d.c);
    if (U_max > kMaxActive) return false;
    const int nmt = (d.Hq / d.Hk * U_max + 127) / 128;
    size_t need;
    switch (d.d) {
        case 16: need = AttSmem<16>(d.T, nmt).total; break;
        case 32: need = AttSmem<32>(d.T, nmt).total; break;
        case 64: need = AttSmem<64>(d.T, nmt).total; break;
        default: return false;
    }
    return need <= 220 * 1024 && (long long)d.B * d.Hk * d.T < 0x7fffffffLL;
}

int launch_attend_tc(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    switch (a.d.d) {
        case 16: return launch_d<16>(ctx, a, st);
        case 32: return launch_d<32>(ctx, a, st);
        case 64: return launch_d<64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

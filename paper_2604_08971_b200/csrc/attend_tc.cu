// SentryAttend (Section 4.4, Eq. 6) for bf16 tensors on the 5th-generation tensor cores, for
// sequences whose K and V rows of one KV group fit in shared memory (T up to ~1.5 k at d = 32).
//
// One CTA per (sample, KV group) does everything for the group's kept heads:
//   1. Present tokens of the sample -> runs of consecutive tokens.  K, V (and later Q) rows sit in
//      shared memory in present-token order, in the swizzled row layout the tensor core reads.
//      The part of every run between 8-row boundaries comes by TMA tensor copies (boxes of 64
//      and of 8 rows, each CTA fetching its own copy); the few rows before and behind it, and everything when the
//      present tokens are scattered over more than kMaxRuns runs, come by 16-byte async copies
//      into the same layout.  K and V are read from HBM once per group.
//   2. Sparsity scores (max minus mean of q.k/sqrt(d) over the sampled keys of every query): one
//      thread per query walks its sampled key rows in shared memory, all kept heads of the group
//      in one pass (fp32 accumulation of exact bf16 products).  Every query has its own sampled
//      keys, so this step is a gather, not a contraction.  (A dense form -- S = Q K^T for all
//      queries on the tensor core, maximum and sum over the sampled keys taken by predicated
//      instructions while reading the accumulator -- was built and measured: it is bound by the
//      half-rate compare/min-max pipe at four of its cycles per (query, key) and lost to the
//      gather on every workload.)
//   3. Top-U selection per head (ties -> lower index).
//   4. Eq. 6 on the active rows: the U rows of all kept heads of the group are stacked into
//      M = 128 row tiles; four softmax warps own one accumulator row per lane.
//        pass 1  S = Q_act K^T in chunks of 256 keys -> row maxima
//        pass 2  per 64-key tile: S again, p = 2^((s - max) c) split into a bf16 head and a bf16
//                remainder (p = p_hi + p_lo to 2^-17), both written back to TENSOR MEMORY
//                and used from there as the A operand of  O += P V,  V read in place from
//                shared memory as an MN-major operand.  The issuer hands over once per tile:
//                P V of tile t and Q K^T of tile t+2 go out together.
//   5. Meanwhile the remaining warps sum the columns of V (the context vector) and write the
//      context rows and the zero rows of absent tokens; the softmax warps finish with O / l.
// Every wait is bounded; on expiry the CTA raises SENTRY_STATUS_BIT_TIMEOUT and unwinds.
#include <cuda.h>

#include "attend_common.cuh"
#include "tc_common.cuh"

namespace {

constexpr int kMaxRuns = 8;         // runs of consecutive present tokens fetched by TMA
constexpr int kKT = 64;             // keys per S tile of Eq. 6, pass 2
constexpr int kChunk = 256;         // keys per S chunk of Eq. 6, pass 1
constexpr int kTmemColsAtt = 256;   // one 256-key chunk, or  S0 | S1 | O | P_hi | P_lo
constexpr int kColS0 = 0, kColS1 = 64, kColO = 128, kColPH = 192, kColPL = 224;
constexpr int kIssuerWarp = 0;      // TMA producer and UMMA issuer
constexpr int kSoftmaxWarp0 = 4;    // warps 4-7 own the accumulator rows (score epilogue, softmax)
constexpr int kThreadsSmall = 256, kThreadsBig = 512;   // warps 1-3 (and 8+): bit rows, context fill

struct AttMisc {
    uint64_t k_full, v_full;
    uint64_t c_full, c_empty;        // Eq. 6 pass 1 chunk
    uint64_t s_full[2];              // Eq. 6 pass 2 S tiles
    uint64_t p_full, p_empty;        // Eq. 6 pass 2 weights in tensor memory
    uint64_t o_full, o_empty;
    uint32_t tmem_base;
    int abort_flag;
    int n_runs;
    int run_p[kMaxRuns + 1];     // first position (in the present-token list) of each run (+ end)
    int fill_next, mean_ready;       // context fill: next block of rows to take; context vector written
    int pick[2];
    int cls[33];
    int wcnt[32];
};

// dynamic shared memory; the kernel carves it in the same order
template <int D>
struct AttSmem {
    static constexpr int RB = D * 2;
    int rows_cap, r_eff;
    size_t off_v, off_q, off_scratch, off_keys, off_misc, off_valid, off_kind, off_abits, total;
    __host__ __device__ AttSmem(int T, int r) {
        rows_cap = (T + kKT - 1) / kKT * kKT;
        r_eff = r < kMaxRK ? r : kMaxRK;
        size_t o = 0;
        o += (size_t)rows_cap * RB;  o = (o + 1023) / 1024 * 1024;  off_v = o;
        o += (size_t)rows_cap * RB;  o = (o + 1023) / 1024 * 1024;  off_q = o;
        o += 2 * (size_t)128 * RB;   o = (o + 1023) / 1024 * 1024;  off_scratch = o;
        o += 8192;   /* selection histograms, then column sums of V */  off_keys = o;
        o += ((size_t)r_eff * T * 4 + 127) / 128 * 128;              off_misc = o;
        o += (sizeof(AttMisc) + 127) / 128 * 128;                    off_valid = o;
        o += ((size_t)T * 2 + 127) / 128 * 128;                      off_kind = o;
        o += ((size_t)T + 127) / 128 * 128;                          off_abits = o;
        o += ((size_t)kMaxRK * ((T + 31) / 32) * 4 + 127) / 128 * 128;
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
// valid-key bits of the 32 keys starting at r0 (keys are the present tokens 0 .. Tv-1)
__device__ __forceinline__ uint32_t key_bits(int r0, int Tv) {
    return r0 + 32 <= Tv ? 0xffffffffu : (r0 < Tv ? (1u << (Tv - r0)) - 1u : 0u);
}

// Rows [w0, w1) of the present-token list (w0 a multiple of 8) of the tensor whose rows of this
// (sample, head) start at global row grow0, into the row buffer at dst (row w0 first).
// tma_part: by ONE thread -- the boxes between the 8-row boundaries inside every run; returns the
// bytes they carry.  edge_part: by `nthr` threads (index `tid`) -- the rows before and behind.
template <int D>
__device__ __forceinline__ uint32_t stage_tma_part(const AttMisc* misc, const uint16_t* s_valid, int n_runs, int w0,
                                                   int w1, uint32_t dst, const CUtensorMap* m64, const CUtensorMap* m8,
                                                   int grow0, uint32_t bar, bool issue) {
    constexpr int RB = D * 2;
    uint32_t bytes = 0;
    for (int k = 0; k < n_runs; ++k) {
        const int p0 = misc->run_p[k], p1 = misc->run_p[k + 1];
        const int a = max(p0, w0), e = min(p1, w1);
        if (a >= e) continue;
        const int m0 = (a + 7) & ~7, m1 = e & ~7;
        if (m1 <= m0) continue;
        bytes += (uint32_t)(m1 - m0) * RB;
        if (issue) {
            const int y0 = grow0 + (int)s_valid[p0] - p0;     // global row of list position 0 of this run
            int r = m0;
            for (; r + 64 <= m1; r += 64) ptx::tma_load_2d(dst + (uint32_t)(r - w0) * RB, m64, 0, y0 + r, bar);
            for (; r < m1; r += 8) ptx::tma_load_2d(dst + (uint32_t)(r - w0) * RB, m8, 0, y0 + r, bar);
        }
    }
    return bytes;
}
template <int D>
__device__ __forceinline__ void stage_edge_part(const AttMisc* misc, const uint16_t* s_valid, int n_runs, int w0, int w1,
                                                uint32_t dst, const __nv_bfloat16* __restrict__ src, int tid, int nthr) {
    using S = Sw<D>;
    if (n_runs == 0) {   // scattered list: every row
        for (int i = tid; i < (w1 - w0) * S::CPR; i += nthr) {
            const int r = w0 + i / S::CPR, cc = i % S::CPR;
            ptx::cp_async_16(dst + S::off(r - w0, cc), src + (size_t)s_valid[r] * D + cc * 8);
        }
        return;
    }
    for (int i = tid; i < n_runs * 14 * S::CPR; i += nthr) {
        const int k = i / (14 * S::CPR), e14 = (i / S::CPR) % 14, cc = i % S::CPR;
        const int p0 = misc->run_p[k], p1 = misc->run_p[k + 1];
        const int a = max(p0, w0), e = min(p1, w1);
        if (a >= e) continue;
        const int m0 = (a + 7) & ~7, m1 = e & ~7;
        const int head_end = min(m0, e), tail_start = max(m1, head_end);
        const int r = e14 < 7 ? a + e14 : tail_start + (e14 - 7);
        const bool in = e14 < 7 ? r < head_end : r < e;
        if (in) ptx::cp_async_16(dst + S::off(r - w0, cc), src + (size_t)s_valid[r] * D + cc * 8);
    }
}

// Sparsity scores of NH heads of the group at once for the queries of this thread, sampled keys
// gathered from the resident K rows (the form for long or scattered lists).  The query rows stay
// in registers as packed bf16, so a sampled key row is fetched once per group.  The 1/sqrt(d) factor
// is applied once at the end (it is positive, so it commutes with the maximum).
template <int D, int NH>
__device__ __forceinline__ void score_pass_gather(const __nv_bfloat16* __restrict__ Q, const size_t* q_base,
                                                  const uint16_t* s_valid, uint32_t ks_addr, int Tv,
                                                  const int32_t* __restrict__ tbl, int n_s, int cnt, int score_mode,
                                                  uint32_t* const* keys_out, unsigned int* status) {
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
        // four are used: a thread walks its own 4 n_s-byte table row, and with most of the L1
        // given to shared memory the row's lines do not survive from one use to the next.
        const int32_t* row = score_mode != 1 ? tbl + (size_t)p * (score_mode == 2 ? 1 : n_s) : nullptr;
        const size_t es = score_mode == 2 ? (size_t)Tv : 1;   // entry-major table: entry a of row p at a * Tv + p
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
                    const float sc = (acc[h][0] + acc[h][1]) + (acc[h][2] + acc[h][3]);
                    mx[h] = fmaxf(mx[h], sc);
                    sum[h] += sc;
                }
            }
        }
#pragma unroll
        for (int h = 0; h < NH; ++h) keys_out[h][p] = sentry_order_key((mx[h] - sum[h] * inv_cnt) * scale);
    }
}

template <int D>
__device__ __forceinline__ void score_heads_gather(const __nv_bfloat16* __restrict__ Q, int b, int Hq, int Tlen, int rk,
                                                const int* hs, const uint16_t* s_valid, uint32_t ks_addr, int Tv,
                                                const int32_t* tbl, int n_s, int cnt, int score_mode,
                                                uint32_t* s_keys, unsigned int* status) {
    constexpr int HPP = (D == 64) ? 2 : 4;   // heads per pass: packed q rows live in registers
    for (int h0 = 0; h0 < rk; h0 += HPP) {
        const int nh = min(HPP, rk - h0);
        size_t q_base[HPP];
        uint32_t* keys_out[HPP];
        for (int j = 0; j < HPP; ++j) {
            const int hh = min(h0 + j, rk - 1);
            q_base[j] = ((size_t)b * Hq + hs[hh]) * Tlen * D;
            keys_out[j] = s_keys + (size_t)hh * Tlen;
        }
#define SCORE_PASS(N) score_pass_gather<D, N>(Q, q_base, s_valid, ks_addr, Tv, tbl, n_s, cnt, score_mode, keys_out, status)
        if (nh == 1) SCORE_PASS(1);
        else if (nh == 2) SCORE_PASS(2);
        else if constexpr (HPP == 4) {
            if (nh == 3) SCORE_PASS(3);
            else SCORE_PASS(4);
        }
#undef SCORE_PASS
    }
}

// grid B*Hk; kThreadsSmall or kThreadsBig threads.  tm_*64 / tm_*8: maps over Q, K and V viewed as
// [B*H*T, D] with boxes of 64 and 8 rows.
template <int D, bool BIG>
__global__ void __launch_bounds__(kThreadsBig, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap tm_k64, const __grid_constant__ CUtensorMap tm_k8,
                 const __grid_constant__ CUtensorMap tm_v64, const __grid_constant__ CUtensorMap tm_v8,
                 const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                 const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ kept_heads,
                 const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks,
                 const int32_t* __restrict__ table, const int64_t* __restrict__ offsets, int n_subsets,
                 const int32_t* __restrict__ active_in, int32_t* __restrict__ active_out, int Tlen, int Hq,
                 int Hk, int k_h, int c, int score_mode, int U_max,
                 __nv_bfloat16* __restrict__ O, unsigned int* status) {
    using S = Sw<D>;
    constexpr int RB = D * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ int red[66];
    __shared__ int32_t s_act[kMaxRK][kMaxActive];
    __shared__ __align__(16) __nv_bfloat16 s_mean[D];

    const uint32_t raw_addr = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw_addr);
    const AttSmem<D> L(Tlen, Hq / Hk);
    const uint32_t ks_addr = base, vs_addr = base + (uint32_t)L.off_v, qs_addr = base + (uint32_t)L.off_q;
    uint8_t* scratch = smem + L.off_scratch;
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(smem + L.off_keys);
    AttMisc* misc = reinterpret_cast<AttMisc*>(smem + L.off_misc);
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(smem + L.off_valid);
    uint8_t* s_kind = smem + L.off_kind;
    uint32_t* s_abits = reinterpret_cast<uint32_t*>(smem + L.off_abits);
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
        ptx::mbar_init(ptx::smem_u32(&misc->c_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->c_empty), 4);
        ptx::mbar_init(ptx::smem_u32(&misc->s_full[0]), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->s_full[1]), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->p_full), 4);
        ptx::mbar_init(ptx::smem_u32(&misc->p_empty), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->o_full), 1);
        ptx::mbar_init(ptx::smem_u32(&misc->o_empty), 4);
        misc->abort_flag = 0;
        misc->fill_next = 0;
        misc->mean_ready = 0;
        ptx::fence_barrier_init();
    }
    if (warp == kIssuerWarp) {
        ptx::tmem_alloc(ptx::smem_u32(&misc->tmem_base), kTmemColsAtt);
        ptx::tmem_relinquish();
    }
    if (warp == 1) {
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
            if (nr > kMaxRuns) nr = 0;      // scattered tokens: every row by 16-byte copies
            misc->run_p[nr] = Tv;
            misc->n_runs = nr;
        }
    }
    for (int t = threadIdx.x; t < Tlen; t += blockDim.x) s_kind[t] = 0;
    for (int i = threadIdx.x; i < kMaxRK * words; i += blockDim.x) s_abits[i] = 0u;
    for (int i = threadIdx.x; i < kMaxRK * kMaxActive; i += blockDim.x) (&s_act[0][0])[i] = -1;
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = misc->tmem_base;
    const int n_runs = misc->n_runs;
    const int n_kt = (Tv + kKT - 1) / kKT;
    const int rows_staged = n_kt * kKT;
    const int grow_kv = (b * Hk + g) * Tlen;
    const __nv_bfloat16* Kg = K + (size_t)grow_kv * D;
    const __nv_bfloat16* Vg = V + (size_t)grow_kv * D;

    // ---- stage K, then V
    if (warp == kIssuerWarp) {
        if (elect_one()) {
            const uint32_t bytes = stage_tma_part<D>(misc, s_valid, n_runs, 0, Tv, 0u, nullptr, nullptr, 0, 0u, false);
            ptx::mbar_arrive_expect_tx(ptx::smem_u32(&misc->k_full), bytes);
            stage_tma_part<D>(misc, s_valid, n_runs, 0, Tv, ks_addr, &tm_k64, &tm_k8, grow_kv,
                              ptx::smem_u32(&misc->k_full), true);
            ptx::mbar_arrive_expect_tx(ptx::smem_u32(&misc->v_full), bytes);
            stage_tma_part<D>(misc, s_valid, n_runs, 0, Tv, vs_addr, &tm_v64, &tm_v8, grow_kv,
                              ptx::smem_u32(&misc->v_full), true);
        }
        __syncwarp();
    }
    stage_edge_part<D>(misc, s_valid, n_runs, 0, Tv, ks_addr, Kg, threadIdx.x, blockDim.x);
    stage_edge_part<D>(misc, s_valid, n_runs, 0, Tv, vs_addr, Vg, threadIdx.x, blockDim.x);
    ptx::cp_async_commit();
    // V rows behind the last present token get weight zero in every softmax, but zero times a stray
    // NaN would still poison a row: clear them
    for (int i = threadIdx.x; i < (rows_staged - Tv) * S::CPR; i += blockDim.x) {
        const int r = Tv + i / S::CPR, cc = i % S::CPR;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vs_addr + S::off(r, cc)), "r"(0) : "memory");
    }
    for (int p = threadIdx.x; p < Tv; p += blockDim.x) s_kind[s_valid[p]] = 1;
    ptx::cp_async_wait_all();
    ptx::fence_proxy_async_smem();   // copied and cleared rows -> visible to the tensor core
    bool ok = __syncthreads_and(warp_wait(&misc->k_full, 0u, abort_flag) ? 1 : 0) != 0;   // block-uniform

    const int n_s = U;
    const int cnt = score_mode != 1 ? n_s : Tv;
    const int32_t* tbl = nullptr;
    bool table_ok = true;
    if (score_mode != 1 && active_in == nullptr) {
        if (mask >= (uint32_t)n_subsets || offsets[mask] < 0) table_ok = false;
        else tbl = table + offsets[mask];
    }

    if (ok && active_in == nullptr && !table_ok) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
        for (int i = threadIdx.x; i < rk * Tlen; i += blockDim.x) s_keys[i] = 0u;
    } else if (ok && active_in == nullptr) {
        // ---- sparsity scores (Section 4.4): every thread walks the sampled key rows of its queries
        score_heads_gather<D>(Q, b, Hq, Tlen, rk, hs, s_valid, ks_addr, Tv, tbl, n_s, cnt, score_mode, s_keys, status);
    }
    ok = __syncthreads_and((ok && *abort_flag == 0) ? 1 : 0) != 0;

    if (ok && active_in == nullptr) {
        // ---- the U present queries with the largest score are active
        int* s_hist = reinterpret_cast<int*>(scratch);
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
    ptx::fence_proxy_async_smem();   // gathered Q rows -> visible to the tensor core
    ok = __syncthreads_and(ok ? 1 : 0) != 0;

    if (!ok) {
        // fall through to the teardown
    } else if (warp == kIssuerWarp) {
        // ------------------------------------------------------------------- UMMA issuer
        constexpr uint32_t idesc_qk = ptx::umma_idesc_bf16(128, kKT);
        constexpr uint32_t idesc_pv = ptx::umma_idesc_bf16_major(128, D, false, true);
        uint32_t nc = 0, np = 0;
        bool iok = true;
        // S[128 x n_keys] = Q_act(tile mt) . K[key0 .. key0 + n_keys)^T into column col
        auto issue_qk = [&](int mt, int key0, uint32_t col, uint32_t idesc) {
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint64_t a = ptx::umma_smem_desc_rows(qs_addr + (uint32_t)mt * 128 * RB + ks * 32, RB);
                const uint64_t bd = ptx::umma_smem_desc_rows(ks_addr + (uint32_t)key0 * RB + ks * 32, RB);
                ptx::umma_bf16(tmem + col, a, bd, idesc, ks > 0 ? 1u : 0u);
            }
        };
        for (int mt = 0; mt < nmt && iok; ++mt) {
            // ---- pass 1: row maxima, 256 keys per hand-over (the chunk covers every column,
            // so the previous tile's O must have been read)
            iok = warp_wait(&misc->o_empty, ((uint32_t)mt & 1u) ^ 1u, abort_flag);
            for (int k0 = 0; k0 < rows_staged && iok; k0 += kChunk) {
                iok = warp_wait(&misc->c_empty, (nc & 1u) ^ 1u, abort_flag);
                if (!iok) break;
                ptx::tc_fence_after_sync();
                if (elect_one()) {
                    issue_qk(mt, k0, 0u, ptx::umma_idesc_bf16(128, min(kChunk, rows_staged - k0)));
                    ptx::umma_commit(ptx::smem_u32(&misc->c_full));
                }
                __syncwarp();
                ++nc;
            }
            if (!iok) break;
            // ---- pass 2: the first two S tiles go out as soon as the last chunk has been read
            iok = warp_wait(&misc->c_empty, (nc & 1u) ^ 1u, abort_flag);
            if (!iok) break;
            ptx::tc_fence_after_sync();
            if (elect_one()) {
                issue_qk(mt, 0, kColS0, idesc_qk);
                ptx::umma_commit(ptx::smem_u32(&misc->s_full[0]));
                if (n_kt > 1) {
                    issue_qk(mt, kKT, kColS1, idesc_qk);
                    ptx::umma_commit(ptx::smem_u32(&misc->s_full[1]));
                }
            }
            __syncwarp();
            for (int t = 0; t < n_kt && iok; ++t) {
                // weights of tile t are in tensor memory (so S of tile t has been read as well)
                iok = warp_wait(&misc->p_full, np & 1u, abort_flag);
                if (!iok) break;
                ++np;
                ptx::tc_fence_after_sync();
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kKT / 16; ++kk) {
                        const uint64_t bd = ptx::umma_smem_desc_rows(vs_addr + (uint32_t)(t * kKT + kk * 16) * RB, RB);
                        ptx::umma_bf16_tmem_a(tmem + kColO, tmem + kColPH + 8 * kk, bd, idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
                        ptx::umma_bf16_tmem_a(tmem + kColO, tmem + kColPL + 8 * kk, bd, idesc_pv, 1u);
                    }
                    ptx::umma_commit(ptx::smem_u32(&misc->p_empty));
                    if (t == n_kt - 1) ptx::umma_commit(ptx::smem_u32(&misc->o_full));
                    if (t + 2 < n_kt) {
                        issue_qk(mt, (t + 2) * kKT, (t & 1) ? kColS1 : kColS0, idesc_qk);
                        ptx::umma_commit(ptx::smem_u32(&misc->s_full[t & 1]));
                    }
                }
                __syncwarp();
            }
        }
    } else if (warp >= kSoftmaxWarp0 && warp < kSoftmaxWarp0 + 4) {
        // ----------------------------------------------------------------- softmax warps
        const int quarter = warp & 3;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const float cl2 = rsqrtf((float)D) * 1.4426950408889634f;   // 1/sqrt(d) * log2(e)
        uint32_t nc = 0, np = 0, nsf[2] = {0u, 0u};
        bool sok = true;
        for (int mt = 0; mt < nmt && sok; ++mt) {
            const int row = mt * 128 + quarter * 32 + lane;
            const bool warp_has_rows = mt * 128 + quarter * 32 < R;
            // ---- pass 1: maximum of the row over the present keys
            float mx0 = -INFINITY, mx1 = -INFINITY;
            for (int k0 = 0; k0 < rows_staged && sok; k0 += kChunk) {
                sok = warp_wait(&misc->c_full, nc & 1u, abort_flag);
                if (!sok) break;
                ++nc;
                ptx::tc_fence_after_sync();
                if (warp_has_rows) {
                    const int n_grp = min(kChunk, rows_staged - k0) / 32;
                    for (int gq = 0; gq < n_grp; ++gq) {
                        uint32_t sv[32];
                        ptx::tmem_ld_32x32(lane_base + 32 * gq, sv);
                        ptx::tmem_ld_wait();
                        const uint32_t kb = key_bits(k0 + 32 * gq, Tv);
                        if (kb == 0xffffffffu) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                mx0 = max3(mx0, __uint_as_float(sv[i]), __uint_as_float(sv[i + 1]));
                                mx1 = max3(mx1, __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if ((kb >> i) & 1u) mx0 = fmaxf(mx0, __uint_as_float(sv[i]));
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                warp_arrive(&misc->c_empty);
            }
            if (!sok) break;
            // ---- pass 2: weights, two bf16 per weight (head and remainder), into tensor memory
            const float shift = -fmaxf(mx0, mx1) * cl2;
            float l0 = 0.f, l1 = 0.f;
            for (int t = 0; t < n_kt && sok; ++t) {
                const uint32_t buf = (uint32_t)t & 1u;
                sok = warp_wait(&misc->s_full[buf], nsf[buf] & 1u, abort_flag);
                if (!sok) break;
                ++nsf[buf];
                ptx::tc_fence_after_sync();
                const uint32_t tcol = lane_base + (buf ? kColS1 : kColS0);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t ph[16], pl[16];
                    if (warp_has_rows) {
                        uint32_t sv[32];
                        ptx::tmem_ld_32x32(tcol + 32 * half, sv);
                        ptx::tmem_ld_wait();
                        const uint32_t kb = key_bits(t * kKT + 32 * half, Tv);
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * i]), cl2, shift));
                            float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * i + 1]), cl2, shift));
                            if (kb != 0xffffffffu) {
                                p0 = ((kb >> (2 * i)) & 1u) ? p0 : 0.f;
                                p1 = ((kb >> (2 * i + 1)) & 1u) ? p1 : 0.f;
                            }
                            l0 += p0;
                            l1 += p1;
                            const uint32_t h = pack2(p0, p1);
                            ph[i] = h;
                            pl[i] = pack2(p0 - __uint_as_float(h << 16), p1 - __uint_as_float(h & 0xffff0000u));
                        }
                    }
                    if (half == 0) {
                        // the tensor core has finished reading the previous tile's weights
                        sok = warp_wait(&misc->p_empty, (np & 1u) ^ 1u, abort_flag);
                        if (!sok) break;
                        ++np;
                        ptx::tc_fence_after_sync();
                    }
                    if (warp_has_rows) {
                        ptx::tmem_st_32x16(lane_base + kColPH + 16 * half, ph);
                        ptx::tmem_st_32x16(lane_base + kColPL + 16 * half, pl);
                    }
                }
                if (!sok) break;
                ptx::tmem_st_wait();
                ptx::tc_fence_before_sync();
                warp_arrive(&misc->p_full);
            }
            if (!sok) break;
            // ---- rows of this tile: O / l -> bf16 -> global
            sok = warp_wait(&misc->o_full, (uint32_t)mt & 1u, abort_flag);
            if (!sok) break;
            ptx::tc_fence_after_sync();
            uint32_t o[D];
            if (warp_has_rows) {
                if constexpr (D == 16) {
                    ptx::tmem_ld_32x16(lane_base + kColO, reinterpret_cast<uint32_t(&)[16]>(o));
                } else {
#pragma unroll
                    for (int j = 0; j < D / 32; ++j)
                        ptx::tmem_ld_32x32(lane_base + kColO + 32 * j, reinterpret_cast<uint32_t(&)[32]>(o[32 * j]));
                }
                ptx::tmem_ld_wait();
            }
            ptx::tc_fence_before_sync();
            warp_arrive(&misc->o_empty);
            if (warp_has_rows && row < R) {
                const int hh = row / UA, a = row - hh * UA;
                const int tkn = s_act[hh][a];
                if (tkn >= 0) {
                    const float inv = 1.0f / (l0 + l1);
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
        // ------------------------------------------------------------------ context vector
        // warps 1-3 and the warps behind the softmax warps: column sums of V
        const int n_fill = (int)blockDim.x - 5 * 32;
        const int ft = warp < kSoftmaxWarp0 ? (int)threadIdx.x - 32 : (int)threadIdx.x - 5 * 32;
        constexpr int DP = D / 2;
        float (*s_vpart)[D] = reinterpret_cast<float (*)[D]>(scratch);      // [n_fill / DP][D], <= 8 KB
        const int vs_dp = ft % DP, vs_k0 = ft / DP;
        const int stride = min(n_fill / DP, 8192 / (D * 4));
        if (vs_k0 < stride) {
            float v0[4] = {0.f, 0.f, 0.f, 0.f}, v1[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t col = (uint32_t)(vs_dp & 3) * 4;
            int r = vs_k0;
            for (; r + 3 * stride < rows_staged; r += 4 * stride) {   // rows behind the last present token are zero
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    uint32_t w;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(vs_addr + S::off(r + u * stride, vs_dp >> 2) + col));
                    v0[u] += __uint_as_float(w << 16);
                    v1[u] += __uint_as_float(w & 0xffff0000u);
                }
            }
            for (; r < rows_staged; r += stride) {
                uint32_t w;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(vs_addr + S::off(r, vs_dp >> 2) + col));
                v0[0] += __uint_as_float(w << 16);
                v1[0] += __uint_as_float(w & 0xffff0000u);
            }
            s_vpart[vs_k0][2 * vs_dp] = (v0[0] + v0[1]) + (v0[2] + v0[3]);
            s_vpart[vs_k0][2 * vs_dp + 1] = (v1[0] + v1[1]) + (v1[2] + v1[3]);
        }
        bar_sync_group(1, n_fill);
        if (ft < D) {
            float t = 0.f;
            for (int i = 0; i < stride; ++i) t += s_vpart[i][ft];
            s_mean[ft] = __float2bfloat16_rn(t / (float)Tv);
        }
        bar_sync_group(1, n_fill);
        if (ft == 0) { __threadfence_block(); *(volatile int*)&misc->mean_ready = 1; }
    }
    // ---- context rows and zero rows (absent tokens), in blocks of 32 tokens per warp: the warps of the
    // fill group start at once, the others join when their own part is done -- if the context vector
    // is there by then; nobody waits for it
    if (ok && (warp < kSoftmaxWarp0 && warp != kIssuerWarp || warp >= kSoftmaxWarp0 + 4 ||
               *(volatile int*)&misc->mean_ready != 0)) {
        __threadfence_block();
        const uint4* mean4 = reinterpret_cast<const uint4*>(s_mean);
        const int blocks_per_head = (Tlen + 31) / 32;
        const int n_items = rk * blocks_per_head;
        for (;;) {
            int item = 0;
            if (lane == 0) item = atomicAdd(&misc->fill_next, 1);
            item = __shfl_sync(0xffffffffu, item, 0);
            if (item >= n_items) break;
            const int hh = item / blocks_per_head, t0 = (item % blocks_per_head) * 32;
            uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * k_h + khs[hh]) * Tlen * D);
            const uint32_t act = s_abits[hh * words + (t0 >> 5)];
            const int n_tok = min(32, Tlen - t0);
#pragma unroll
            for (int j = 0; j < S::CPR; ++j) {
                const int i = j * 32 + lane;                 // piece of the block: token i / CPR, chunk i % CPR
                const int tl = i / S::CPR, cc = i % S::CPR;
                if (tl < n_tok && !((act >> tl) & 1u))
                    dst[(size_t)(t0 + tl) * S::CPR + cc] = s_kind[t0 + tl] ? mean4[cc] : make_uint4(0, 0, 0, 0);
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
    if (warp == kIssuerWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, kTmemColsAtt);
    }
}

template <int D>
int launch_d(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    const sentry_attend_desc& d = a.d;
    const AttSmem<D> L(d.T, d.Hq / d.Hk);
    const uint64_t kv_rows = (uint64_t)d.B * d.Hk * d.T;
    CUtensorMap k64, k8, v64, v8;
    if (!make_map_2d(&k64, a.K, kv_rows, D, 64, D) || !make_map_2d(&k8, a.K, kv_rows, D, 8, D) ||
        !make_map_2d(&v64, a.V, kv_rows, D, 64, D) || !make_map_2d(&v8, a.V, kv_rows, D, 8, D))
        return SENTRY_ERR_CUDA;
    // two CTAs per SM (each holds 256 of the 512 tensor-memory columns) when the rows fit twice,
    // else one larger CTA
    const bool big = L.total > 106 * 1024;
    size_t smem = L.total;
    if (!big && smem < 80 * 1024) smem = 80 * 1024;   // never more than two CTAs per SM
    LaunchScope ls(ctx, KS_ATT_CORE, st);
    if (big) {
        auto kern = attend_tc_kernel<D, true>;
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        kern<<<d.B * d.Hk, kThreadsBig, smem, st>>>(
            k64, k8, v64, v8, (const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K, (const __nv_bfloat16*)a.V,
            a.kept_heads, a.ids, a.masks, a.sample_table, a.sample_offsets, a.n_subsets,
            a.selection_given ? a.active : nullptr, a.selection_given ? nullptr : a.active_out_user, d.T, d.Hq, d.Hk,
            d.k_h, d.c, d.score_mode, a.U_max, (__nv_bfloat16*)a.O, a.status);
    } else {
        auto kern = attend_tc_kernel<D, false>;
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        kern<<<d.B * d.Hk, kThreadsSmall, smem, st>>>(
            k64, k8, v64, v8, (const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K, (const __nv_bfloat16*)a.V,
            a.kept_heads, a.ids, a.masks, a.sample_table, a.sample_offsets, a.n_subsets,
            a.selection_given ? a.active : nullptr, a.selection_given ? nullptr : a.active_out_user, d.T, d.Hq, d.Hk,
            d.k_h, d.c, d.score_mode, a.U_max, (__nv_bfloat16*)a.O, a.status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

}  // namespace

// bf16, at most kMaxRK query heads per KV group, U <= kMaxActive, and K, V of a group (plus the
// working buffers) within the shared memory of one SM.
bool attend_tc_supported(const sentry_attend_desc& d) {
    if (d.dtype != SENTRY_BF16) return false;
    if (d.Hq / d.Hk > kMaxRK) return false;
    if (sentry_num_active(d.T, d.c) > kMaxActive) return false;
    size_t need;
    switch (d.d) {
        case 16: need = AttSmem<16>(d.T, d.Hq / d.Hk).total; break;
        case 32: need = AttSmem<32>(d.T, d.Hq / d.Hk).total; break;
        case 64: need = AttSmem<64>(d.T, d.Hq / d.Hk).total; break;
        default: return false;
    }
    return need <= 220 * 1024 && (long long)d.B * d.Hq * d.T < 0x7fffffffLL;
}

int launch_attend_tc(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    switch (a.d.d) {
        case 16: return launch_d<16>(ctx, a, st);
        case 32: return launch_d<32>(ctx, a, st);
        case 64: return launch_d<64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

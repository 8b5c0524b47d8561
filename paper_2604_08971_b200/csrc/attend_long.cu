// SentryAttend query selection (Section 4.4) for sequences whose K and V do not fit in shared
// memory together: sparsity scores and the top-U selection of one (sample, KV group) in one CTA,
// with the group's present K rows resident in shared memory -- all of them when they fit beside
// the score arrays (T_v up to ~2.8 k at d = 32), otherwise in a few equal segments that every
// query walks in turn.  The K rows of a group are staged once per segment for ALL its queries;
// the active lists go to global memory and the streamed Eq. 6 kernel takes them from there.
#include "attend_common.cuh"

namespace {

constexpr int kLongThreads = 512;

// Scores of NH heads for the queries of this thread against the segment [seg0, seg0 + seg_n) of
// present keys held at ks_addr.  With one segment the order keys go straight to keys[h][p]; with
// several, running maxima (in keys[], as floats) and sums (sums[]) are carried from segment to
// segment and the last one writes the order keys.
template <int D, int NH>
__device__ __forceinline__ void long_score_segment(const __nv_bfloat16* __restrict__ Q, const size_t* q_base,
                                                   const uint16_t* s_valid, uint32_t ks_addr, int Tv, int seg0,
                                                   int seg_n, bool first, bool last, const int32_t* __restrict__ tbl,
                                                   int n_s, int cnt, int score_mode, uint32_t* const* keys,
                                                   float* const* sums, unsigned int* status) {
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
        for (int h = 0; h < NH; ++h) {
            mx[h] = first ? -INFINITY : __uint_as_float(keys[h][p]);
            sum[h] = first ? 0.f : sums[h][p];
        }
        if (score_mode != 1) {
            // sampled positions, requested four ahead of their use.  Query-major table: entry a of
            // row p at p * n_s + a; entry-major (score_mode 2): a * Tv + p
            const int32_t* row = tbl + (size_t)p * (score_mode == 2 ? 1 : n_s);
            const size_t es = score_mode == 2 ? (size_t)Tv : 1;
            int nxt[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) nxt[u] = __ldg(row + (size_t)min(u, cnt - 1) * es);
            for (int a0 = 0; a0 < cnt; a0 += 4) {
                int cur[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    cur[u] = nxt[u];
                    nxt[u] = __ldg(row + (size_t)min(a0 + 4 + u, cnt - 1) * es);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (a0 + u >= cnt) break;
                    int pj = cur[u];
                    if (pj < 0 || pj >= Tv) { if (first) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); pj = 0; }
                    const int r = pj - seg0;
                    if (r >= 0 && r < seg_n) score_one_key<D, NH>(qw, ks_addr, r, scale, mx, sum);
                }
            }
        } else {
            for (int r = 0; r < seg_n; ++r) score_one_key<D, NH>(qw, ks_addr, r, scale, mx, sum);
        }
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            if (last) keys[h][p] = sentry_order_key(mx[h] - sum[h] * inv_cnt);
            else { keys[h][p] = __float_as_uint(mx[h]); sums[h][p] = sum[h]; }
        }
    }
}

// grid B*Hk, kLongThreads threads, one CTA per SM.  Dynamic shared memory (smem_bytes in all):
//   valid[T] u16 | hist[kMaxRK][256] | keys[rk][T_v] u32 | (several segments: sums[rk][T_v] f32) | K segment
template <int D>
__global__ void __launch_bounds__(kLongThreads, 1)
attend_long_select_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                          const int32_t* __restrict__ kept_heads, const int32_t* __restrict__ ids,
                          const uint32_t* __restrict__ masks, const int32_t* __restrict__ table,
                          const int64_t* __restrict__ offsets, int n_subsets, int Tlen, int Hq, int Hk,
                          int k_h, int c, int score_mode, int U_max, int smem_bytes,
                          int32_t* __restrict__ active, unsigned int* status) {
    using S = Sw<D>;
    extern __shared__ __align__(128) uint8_t s_raw[];
    __shared__ int red[66];
    __shared__ int32_t s_act[kMaxRK][kMaxActive];
    const int b = blockIdx.x / Hk, g = blockIdx.x % Hk;
    const uint32_t mask = masks[b];
    size_t o = 0;
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(s_raw);   o += (((size_t)Tlen * 2 + 127) / 128) * 128;
    int* s_hist = reinterpret_cast<int*>(s_raw + o);           o += (size_t)kMaxRK * 256 * 4;
    const int Tv = block_build_valid(ids, Tlen, mask, s_valid, red);
    int hs[kMaxRK], khs[kMaxRK];
    bool bad;
    const int rk = group_heads(kept_heads + (size_t)b * k_h, k_h, Hq / Hk, g, Hq, hs, khs, bad);
    if (bad && threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
    if (rk == 0) return;
    if (Tv == 0) {   // the Eq. 6 kernel zeroes the rows and raises the flag
        for (int i = threadIdx.x; i < rk * U_max; i += blockDim.x)
            active[((size_t)b * k_h + khs[i / U_max]) * U_max + i % U_max] = -1;
        return;
    }
    const int U = sentry_num_active(Tv, c);
    const int n_s = U;
    const int cnt = score_mode != 1 ? n_s : Tv;
    const int32_t* tbl = nullptr;
    bool table_ok = true;
    if (score_mode != 1) {
        if (mask >= (uint32_t)n_subsets || offsets[mask] < 0) table_ok = false;
        else tbl = table + offsets[mask];
    }
    // segments: everything at once if the rows fit beside the keys, else equal parts beside keys and sums
    const size_t arr = (((size_t)rk * Tv * 4 + 127) / 128) * 128;
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_raw + o);
    const long long room1 = (long long)smem_bytes - (long long)o - (long long)arr;
    int n_seg = 1, seg_rows = Tv;
    float* s_sums = nullptr;
    size_t k_off = o + arr;
    if ((long long)Tv * S::RB > room1) {
        s_sums = reinterpret_cast<float*>(s_raw + o + arr);
        k_off = o + 2 * arr;
        const long long room2 = room1 - (long long)arr;
        const int cap = (int)((room2 > 0 ? room2 : 0) / S::RB) & ~7;
        if (cap < 64) {   // the host sizes the launch so that this cannot happen
            if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            table_ok = false;
        } else {
            n_seg = (Tv + cap - 1) / cap;
            seg_rows = ((Tv + n_seg - 1) / n_seg + 7) & ~7;
        }
    }
    const uint32_t ks_addr = ptx::smem_u32(s_raw + k_off);
    const __nv_bfloat16* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    for (int i = threadIdx.x; i < kMaxRK * kMaxActive; i += blockDim.x) (&s_act[0][0])[i] = -1;

    if (table_ok) {
        for (int sg = 0; sg < n_seg; ++sg) {
            const int seg0 = sg * seg_rows, seg_n = min(seg_rows, Tv - seg0);
            __syncthreads();   // the previous segment is no longer being read
            for (int i = threadIdx.x; i < seg_n * S::CPR; i += blockDim.x) {
                const int row = i / S::CPR, cc = i % S::CPR;
                ptx::cp_async_16(ks_addr + S::off(row, cc), Kg + (size_t)s_valid[seg0 + row] * D + cc * 8);
            }
            ptx::cp_async_wait_all();
            __syncthreads();
            constexpr int HPP = (D == 64) ? 2 : 4;   // heads per pass: packed q rows live in registers
            for (int h0 = 0; h0 < rk; h0 += HPP) {
                const int nh = min(HPP, rk - h0);
                size_t q_base[4];
                uint32_t* keys_h[4];
                float* sums_h[4];
                for (int j = 0; j < 4; ++j) {
                    const int hh = min(h0 + j, rk - 1);
                    q_base[j] = ((size_t)b * Hq + hs[hh]) * Tlen * D;
                    keys_h[j] = s_keys + (size_t)hh * Tv;
                    sums_h[j] = s_sums ? s_sums + (size_t)hh * Tv : nullptr;
                }
#define LONG_SEG(N) long_score_segment<D, N>(Q, q_base, s_valid, ks_addr, Tv, seg0, seg_n, sg == 0, sg == n_seg - 1, \
                                             tbl, n_s, cnt, score_mode, keys_h, sums_h, status)
                if (nh == 1) LONG_SEG(1);
                else if (nh == 2) LONG_SEG(2);
                else if constexpr (HPP == 4) {
                    if (nh == 3) LONG_SEG(3);
                    else LONG_SEG(4);
                }
#undef LONG_SEG
            }
        }
    } else {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
        for (int i = threadIdx.x; i < rk * Tv; i += blockDim.x) s_keys[i] = 0u;
    }
    __syncthreads();
    // ---- the U present queries with the largest score are active (ties -> lower index)
    if (Tv <= 256) warps_select_topk_heads(s_keys, Tv, Tv, U, rk, s_act, s_valid);
    else block_select_topk_heads(s_keys, Tv, Tv, U, rk, s_act, s_valid, s_hist);
    __syncthreads();
    for (int i = threadIdx.x; i < rk * U_max; i += blockDim.x) {
        const int hh = i / U_max, a = i % U_max;
        active[((size_t)b * k_h + khs[hh]) * U_max + a] = a < U ? s_act[hh][a] : -1;
    }
}

template <int D>
size_t long_fixed_bytes(int T) { return (((size_t)T * 2 + 127) / 128) * 128 + (size_t)kMaxRK * 256 * 4; }

constexpr size_t kLongSmemMax = 220 * 1024;

template <int D>
bool long_fits(const sentry_attend_desc& d) {
    // worst case: every head of a group kept and every token present, split into segments
    int rk = d.Hq / d.Hk;
    if (rk > kMaxRK) rk = kMaxRK;
    if (rk > d.k_h) rk = d.k_h;
    const size_t arr = (((size_t)rk * d.T * 4 + 127) / 128) * 128;
    return long_fixed_bytes<D>(d.T) + 2 * arr + (size_t)128 * D * 2 <= kLongSmemMax;
}

template <int D>
int launch_long_d(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    const sentry_attend_desc& d = a.d;
    int rk = d.Hq / d.Hk;
    if (rk > kMaxRK) rk = kMaxRK;
    if (rk > d.k_h) rk = d.k_h;
    // everything resident if the worst case allows it, else all the shared memory there is
    size_t smem = long_fixed_bytes<D>(d.T) + (((size_t)rk * d.T * 4 + 127) / 128) * 128 + (size_t)((d.T + 7) & ~7) * D * 2;
    if (smem > kLongSmemMax) smem = kLongSmemMax;
    auto kern = attend_long_select_kernel<D>;
    SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    LaunchScope ls(ctx, KS_ATT_SCORE, st);
    kern<<<d.B * d.Hk, kLongThreads, smem, st>>>(
        (const __nv_bfloat16*)a.Q, (const __nv_bfloat16*)a.K, a.kept_heads, a.ids, a.masks, a.sample_table,
        a.sample_offsets, a.n_subsets, d.T, d.Hq, d.Hk, d.k_h, d.c, d.score_mode, a.U_max, (int)smem, a.active, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

}  // namespace

// Whether the one-CTA-per-group selection kernel can take the shape (the caller falls back to the
// query-block score kernel otherwise).
bool attend_long_select_supported(const sentry_attend_desc& d) {
    switch (d.d) {
        case 16: return long_fits<16>(d);
        case 32: return long_fits<32>(d);
        case 64: return long_fits<64>(d);
        default: return false;
    }
}

int launch_attend_long_select(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    switch (a.d.d) {
        case 16: return launch_long_d<16>(ctx, a, st);
        case 32: return launch_long_d<32>(ctx, a, st);
        case 64: return launch_long_d<64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

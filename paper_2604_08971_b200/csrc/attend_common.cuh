// Device helpers shared by the bf16 SentryAttend kernels (Section 4.4): the swizzled row layout of
// K/V in shared memory, the sampled-score arithmetic and the top-U selections.
#pragma once
#include <math.h>

#include "common.cuh"
#include "ptx/sm100.cuh"

// The kernels that include this header exist twice: for bf16 tensors, and -- compiled again with
// SENTRY_ATT_F16 defined, under other entry-point names (attend_f16.cu, attend_long_f16.cu) -- for
// IEEE-half tensors.  The two builds differ only in the helpers below: the operand type of the
// mixed-precision FMA and of the warp MMA, and the 16-bit packing / unpacking.
#ifdef SENTRY_ATT_F16
#define ATT_PTX_TYPE "f16"
#define ATT_DTYPE SENTRY_F16
#else
#define ATT_PTX_TYPE "bf16"
#define ATT_DTYPE SENTRY_BF16
#endif

namespace {

// Low / high element of a packed 16-bit pair as fp32, and fp32 -> the 16 storage bits.
__device__ __forceinline__ float att_lo(uint32_t w) {
#ifdef SENTRY_ATT_F16
    return __half2float(__ushort_as_half((unsigned short)(w & 0xffffu)));
#else
    return __uint_as_float(w << 16);
#endif
}
__device__ __forceinline__ float att_hi(uint32_t w) {
#ifdef SENTRY_ATT_F16
    return __half2float(__ushort_as_half((unsigned short)(w >> 16)));
#else
    return __uint_as_float(w & 0xffff0000u);
#endif
}
__device__ __forceinline__ unsigned short att_bits(float x) {
#ifdef SENTRY_ATT_F16
    return __half_as_ushort(__float2half_rn(x));
#else
    return __bfloat16_as_ushort(__float2bfloat16_rn(x));
#endif
}

constexpr int kMaxRK = 4;          // kept heads of one KV group handled per CTA
constexpr int kScoreThreads = 256;
constexpr int kCoreThreads = 256;
constexpr int kCoreWarps = kCoreThreads / 32;
constexpr int kKeyTile = 64;
constexpr int kMaxActive = 48;
constexpr int kSmallT = 256;   // fused attention: sequences up to this length run in 128-thread CTAs
constexpr int kOrderMaxBatch = 1024; // batches up to this size are walked heaviest-sample-first     // U <= 45 for T <= 8103 with c = 5 (checked on the host)

// Row layout in shared memory: rows of D bf16, 16-byte chunks XOR-swizzled so that both
// 8-consecutive-row matrix loads and random row gathers spread over the banks.
template <int D>
struct Sw {
    static constexpr int RB = D * 2;          // row bytes
    static constexpr int CPR = RB / 16;       // 16-byte chunks per row
    static constexpr int RPL = 128 / RB;      // rows per 128-byte line (>= 1 for D <= 64)
    __device__ static __forceinline__ uint32_t off(int row, int c) {
        return (uint32_t)row * RB + (uint32_t)((c ^ ((row / RPL) & (CPR - 1))) << 4);
    }
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Kept heads of KV group g among kept_heads[b, :]: their head ids and kept-list slots.
__device__ __forceinline__ int group_heads(const int32_t* kept, int k_h, int r, int g, int Hq,
                                           int (&hs)[kMaxRK], int (&khs)[kMaxRK], bool& bad) {
    int rk = 0;
    bad = false;
    for (int j = 0; j < k_h; ++j) {
        const int h = kept[j];
        if (h < 0 || h >= Hq) { bad = true; continue; }
        if (h / r == g && rk < kMaxRK) { hs[rk] = h; khs[rk] = j; ++rk; }
    }
    return rk;
}

// ------------------------------------------------------------------------------------ score
// acc_lo += a.lo * b.lo, acc_hi += a.hi * b.hi for two bf16 pairs, in fp32: the mixed-precision
// FMA of sm_100 takes the bf16 operands as they are (exact products, fp32 accumulate), so
// neither the query nor the key row has to be unpacked to fp32 first.
__device__ __forceinline__ void fma_bf16_pair(float& acc_lo, float& acc_hi, uint32_t a, uint32_t b) {
    asm("{\n\t.reg .b16 al, ah, bl, bh;\n\t"
        "mov.b32 {al, ah}, %2;\n\tmov.b32 {bl, bh}, %3;\n\t"
        "fma.rn.f32." ATT_PTX_TYPE " %0, al, bl, %0;\n\tfma.rn.f32." ATT_PTX_TYPE " %1, ah, bh, %1;\n\t}"
        : "+f"(acc_lo), "+f"(acc_hi)
        : "r"(a), "r"(b));
}

// s = q . k / sqrt(d) for NH heads against one key row in shared memory; updates max and sum.
template <int D, int NH>
__device__ __forceinline__ void score_one_key(const uint32_t (&qw)[NH][D / 2], uint32_t row_addr_base, int row,
                                              float scale, float (&mx)[NH], float (&sum)[NH]) {
    using S = Sw<D>;
    float acc[NH][4];
#pragma unroll
    for (int h = 0; h < NH; ++h) acc[h][0] = acc[h][1] = acc[h][2] = acc[h][3] = 0.f;
#pragma unroll
    for (int cc = 0; cc < S::CPR; ++cc) {
        const uint4 v = lds128(row_addr_base + S::off(row, cc));
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

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
#ifdef SENTRY_ATT_F16
    __half2 v = __floats2half2_rn(lo, hi);
#else
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
#endif
    return *reinterpret_cast<uint32_t*>(&v);
}
// bf16 pair of what the packed pair `head` = pack2(lo, hi) leaves of lo and hi
__device__ __forceinline__ uint32_t pack2_rem(float lo, float hi, uint32_t head) {
    return pack2(lo - att_lo(head), hi - att_hi(head));
}

// Warp-level top-k by radix selection over n order keys in shared memory (larger key first,
// ties -> lower index).  Writes remap[index] of the selected entries to out[0..k) in ascending
// index order.  `hist` = 256 ints of shared memory owned by this warp.
__device__ inline void warp_select_topk_radix(const uint32_t* keys, int n, int k, int32_t* out,
                                              const uint16_t* remap, int* hist) {
    const int lane = threadIdx.x & 31;
    uint32_t prefix = 0, fixed = 0;
    int want = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = lane; i < 256; i += 32) hist[i] = 0;
        __syncwarp();
        for (int i = lane; i < n; i += 32) {
            const uint32_t key = keys[i];
            if ((key & fixed) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
        }
        __syncwarp();
        const int top = 255 - 8 * lane;      // this lane's digits, descending
        int mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) mine += hist[top - j];
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int above = incl - mine;
        const bool here = above < want && want <= incl;
        int digit = 0, rem = 0;
        if (here) {
            int acc = above;
            for (int j = 0; j < 8; ++j) {
                const int cdig = hist[top - j];
                if (want <= acc + cdig) { digit = top - j; rem = want - acc; break; }
                acc += cdig;
            }
        }
        const unsigned who = __ballot_sync(0xffffffffu, here);
        const int src = __ffs(who) - 1;
        digit = __shfl_sync(0xffffffffu, digit, src);
        rem = __shfl_sync(0xffffffffu, rem, src);
        prefix |= (uint32_t)digit << shift;
        fixed |= 255u << shift;
        want = rem;
        __syncwarp();
    }
    const uint32_t t = prefix;
    const int need_eq = want;
    int base = 0, eq_seen = 0;
    for (int i0 = 0; i0 < n; i0 += 32) {
        const int i = i0 + lane;
        const uint32_t key = i < n ? keys[i] : 0u;
        const bool is_eq = i < n && key == t, is_gt = i < n && key > t;
        const unsigned em = __ballot_sync(0xffffffffu, is_eq);
        const bool keep = is_gt || (is_eq && eq_seen + __popc(em & ((1u << lane) - 1u)) < need_eq);
        const unsigned km = __ballot_sync(0xffffffffu, keep);
        if (keep) out[base + __popc(km & ((1u << lane) - 1u))] = (int32_t)remap[i];
        base += __popc(km);
        eq_seen += __popc(em);
    }
    __syncwarp();
}

// Top-k of n <= 32 * KPL order keys by ONE warp with the keys in registers (lane l holds keys
// l, l + 32, ...): the k-th largest key is built bit by bit from the top (a candidate bit stays
// set if at least k keys are >= the candidate: 32 steps of KPL compares and one warp add), then
// the entries above it and the first ties are compacted in ascending index order.  No shared-
// memory histograms, no atomics and no block barriers.
template <int KPL>
__device__ __forceinline__ void warp_select_topk_bits(const uint32_t* keys, int n, int k, int32_t* out,
                                                      const uint16_t* remap) {
    const int lane = threadIdx.x & 31;
    uint32_t r[KPL];
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        const int i = j * 32 + lane;
        r[j] = i < n ? keys[i] : 0u;     // padding: below every candidate (candidates are >= 1)
    }
    uint32_t t = 0;
#pragma unroll 1
    for (int b = 31; b >= 0; --b) {
        const uint32_t cand = t | (1u << b);
        int cnt = 0;
#pragma unroll
        for (int j = 0; j < KPL; ++j) cnt += (r[j] >= cand) ? 1 : 0;
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (cnt >= k) t = cand;
    }
    // t is the k-th largest key (0 only if fewer than k keys are non-zero: then every entry ties)
    int gt = 0;
#pragma unroll
    for (int j = 0; j < KPL; ++j) gt += (r[j] > t) ? 1 : 0;
    gt = __reduce_add_sync(0xffffffffu, gt);
    const int need_eq = k - gt;
    int base = 0, eq_seen = 0;
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
        if (j * 32 >= n) break;          // warp-uniform
        const int i = j * 32 + lane;
        const bool is_eq = i < n && r[j] == t, is_gt = i < n && r[j] > t;
        const unsigned em = __ballot_sync(0xffffffffu, is_eq);
        const bool keep = is_gt || (is_eq && eq_seen + __popc(em & ((1u << lane) - 1u)) < need_eq);
        const unsigned km = __ballot_sync(0xffffffffu, keep);
        if (keep) out[base + __popc(km & ((1u << lane) - 1u))] = (int32_t)remap[i];
        base += __popc(km);
        eq_seen += __popc(em);
    }
    __syncwarp();
}
// Warp hh selects for head hh (keys [rk][stride], n <= 256 per head).
__device__ __forceinline__ void warps_select_topk_heads(const uint32_t* keys, int stride, int n, int k, int rk,
                                                        int32_t (*out)[kMaxActive], const uint16_t* remap) {
    const int warp = threadIdx.x >> 5;
    if (warp < rk) warp_select_topk_bits<8>(keys + (size_t)warp * stride, n, k, out[warp], remap);
}
// The same selection for the rk <= kMaxRK heads of a group at once, by the whole block: all
// threads count digits for every head (the long part), warp hh then picks head hh's digit, and
// at the end compacts head hh's selection.  keys: [rk][stride] order keys, n per head;
// hist: kMaxRK * 256 ints of shared memory.
__device__ inline void block_select_topk_heads(const uint32_t* keys, int stride, int n, int k, int rk,
                                               int32_t (*out)[kMaxActive], const uint16_t* remap, int* hist) {
    __shared__ uint32_t s_sel[2 * kMaxRK];   // per head: fixed key prefix, entries still wanted
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < rk) { s_sel[2 * threadIdx.x] = 0u; s_sel[2 * threadIdx.x + 1] = (uint32_t)k; }
    uint32_t fixed = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < rk * 256; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        for (int hh = 0; hh < rk; ++hh) {
            const uint32_t prefix = s_sel[2 * hh];
            const uint32_t* kh = keys + (size_t)hh * stride;
            int* hh_hist = hist + hh * 256;
            for (int i = threadIdx.x; i < n; i += blockDim.x) {
                const uint32_t key = kh[i];
                if ((key & fixed) == prefix) atomicAdd(&hh_hist[(key >> shift) & 255u], 1);
            }
        }
        __syncthreads();
        if (warp < rk) {
            const int* h = hist + warp * 256;
            const int want = (int)s_sel[2 * warp + 1];
            const int top = 255 - 8 * lane;      // this lane's digits, descending
            int mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += h[top - j];
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const int above = incl - mine;
            if (above < want && want <= incl) {   // exactly one lane
                int acc = above;
                for (int j = 0; j < 8; ++j) {
                    const int cdig = h[top - j];
                    if (want <= acc + cdig) {
                        s_sel[2 * warp] |= (uint32_t)(top - j) << shift;
                        s_sel[2 * warp + 1] = (uint32_t)(want - acc);
                        break;
                    }
                    acc += cdig;
                }
            }
        }
        fixed |= 255u << shift;
        __syncthreads();
    }
    if (warp < rk) {
        const uint32_t* kh = keys + (size_t)warp * stride;
        const uint32_t t = s_sel[2 * warp];
        const int need_eq = (int)s_sel[2 * warp + 1];
        int base = 0, eq_seen = 0;
        for (int i0 = 0; i0 < n; i0 += 32) {
            const int i = i0 + lane;
            const uint32_t key = i < n ? kh[i] : 0u;
            const bool is_eq = i < n && key == t, is_gt = i < n && key > t;
            const unsigned em = __ballot_sync(0xffffffffu, is_eq);
            const bool keep = is_gt || (is_eq && eq_seen + __popc(em & ((1u << lane) - 1u)) < need_eq);
            const unsigned km = __ballot_sync(0xffffffffu, keep);
            if (keep) out[warp][base + __popc(km & ((1u << lane) - 1u))] = (int32_t)remap[i];
            base += __popc(km);
            eq_seen += __popc(em);
        }
    }
}

}  // namespace

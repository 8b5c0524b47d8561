// Sparse-MoE block with expert-internal channel pruning (Section 4.6): the routing (which experts a
// token goes to, with which weights) is given and untouched; every expert e runs the compacted pair
// GELU(x W1_e[:, N_e]) W2_e[N_e, :] on the tokens routed to it, and a token's output is the
// weighted sum over its routing slots.
//
// On the device this is the channel-compacted FFN with one kept-channel list AND one weight pair
// per expert:  the (token, slot) pairs are regrouped by expert into the same row plan the dense FFN
// uses (list = expert), with a second row table that sends each result to its own (token, slot)
// row of a staging buffer; the fused-pair kernels run unchanged on that plan; a last kernel forms
// the weighted sum per token in slot order (fp32 accumulation, no atomics on data, so the result
// does not depend on how the rows were grouped).
#include "ffn_plan.cuh"

namespace {

constexpr int kPlanThreads = 256;

// phase 0: counts[e] += routed slots of expert e.   phase 1: reserve, per block, a range of every
// expert's rows (one global atomic per expert and block) and write rowidx / rowout.
// Slot with id -1: not routed (skipped).  Any other id outside [0, E): status bit, skipped.
__global__ void __launch_bounds__(kPlanThreads)
moe_route_kernel(const int32_t* __restrict__ expert_ids, long long n_slots, int E, int top_k, int phase,
                 int32_t* __restrict__ counts, int32_t* __restrict__ cursor, FfnPlan plan, unsigned int* status) {
    extern __shared__ int s_int[];
    int* s_cnt = s_int;        // [E] slots of this block per expert
    int* s_base = s_int + E;   // [E] first position of this block's range in the expert's rows
    for (int e = threadIdx.x; e < E; e += blockDim.x) s_cnt[e] = 0;
    __syncthreads();
    const long long per_block = (long long)kPlanThreads * 8;
    const long long i0 = (long long)blockIdx.x * per_block;
    int my_e[8], my_pos[8];
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const long long i = i0 + (long long)j * kPlanThreads + threadIdx.x;
        my_e[j] = i < n_slots ? __ldg(expert_ids + i) : -1;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        int e = my_e[j];
        if (e < -1 || e >= E) {
            atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            e = -1;
        }
        my_e[j] = e;
        // one shared-memory atomic per (warp, expert): the lanes of a warp that go to the same
        // expert take consecutive positions from their first lane's reservation
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        const int leader = __ffs(peers) - 1;
        int base = 0;
        if (lane == leader && e >= 0) base = atomicAdd(&s_cnt[e], __popc(peers));
        my_pos[j] = __shfl_sync(0xffffffffu, base, leader) + __popc(peers & ((1u << lane) - 1u));
    }
    __syncthreads();
    if (phase == 0) {
        for (int e = threadIdx.x; e < E; e += blockDim.x)
            if (s_cnt[e] > 0) atomicAdd(&counts[e], s_cnt[e]);
        return;
    }
    for (int e = threadIdx.x; e < E; e += blockDim.x)
        s_base[e] = s_cnt[e] > 0 ? plan.list_row0[e] + atomicAdd(&cursor[e], s_cnt[e]) : 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (my_e[j] < 0) continue;
        const long long i = i0 + (long long)j * kPlanThreads + threadIdx.x;
        const int pos = s_base[my_e[j]] + my_pos[j];
        plan.rowidx[pos] = (int32_t)(i / top_k);   // row of X: the token
        plan.rowout[pos] = (int32_t)i;             // row of the staging buffer: (token, slot)
    }
}

// counts -> list_row0, tile_start (exclusive prefix sums over the experts); cursor := 0.
__global__ void __launch_bounds__(kPlanThreads)
moe_offsets_kernel(const int32_t* __restrict__ counts, int E, int tile_rows, FfnPlan plan,
                   int32_t* __restrict__ cursor) {
    __shared__ int s_rows[kPlanThreads], s_tiles[kPlanThreads];
    const int per = (E + kPlanThreads - 1) / kPlanThreads;
    const int e0 = threadIdx.x * per, e1 = min(E, e0 + per);
    int rows = 0, tiles = 0;
    for (int e = e0; e < e1; ++e) {
        rows += counts[e];
        tiles += (counts[e] + tile_rows - 1) / tile_rows;
        cursor[e] = 0;
    }
    s_rows[threadIdx.x] = rows;
    s_tiles[threadIdx.x] = tiles;
    __syncthreads();
    int row0 = 0, tile0 = 0;
    for (int i = 0; i < (int)threadIdx.x; ++i) { row0 += s_rows[i]; tile0 += s_tiles[i]; }
    for (int e = e0; e < e1; ++e) {
        plan.list_row0[e] = row0;
        plan.tile_start[e] = tile0;
        row0 += counts[e];
        tile0 += (counts[e] + tile_rows - 1) / tile_rows;
    }
    if (threadIdx.x == kPlanThreads - 1) {
        plan.list_row0[E] = row0;
        plan.tile_start[E] = tile0;
    }
}

// The whole plan in ONE launch by one block, for small calls (latency: one launch instead of a
// memset and three): count per expert in shared memory, prefix sums, then a second walk that hands
// out the positions (one shared-memory atomic per warp and expert in both walks).
constexpr int kPlanOneThreads = 1024;
constexpr long long kPlanOneMaxSlots = 8192;   // one round of the block; beyond it one SM is the slower way (65 536 slots: 53 us)
__global__ void __launch_bounds__(kPlanOneThreads)
moe_plan_one_kernel(const int32_t* __restrict__ expert_ids, int n_slots, int E, int top_k, int tile_rows,
                    FfnPlan plan, unsigned int* status) {
    extern __shared__ int s_int[];
    int* s_cnt = s_int;          // [E] slots per expert
    int* s_cur = s_int + E;      // [E] next free row of the expert
    const int lane = threadIdx.x & 31;
    for (int e = threadIdx.x; e < E; e += blockDim.x) s_cnt[e] = 0;
    __syncthreads();
    bool bad = false;
    const int per_round = (int)blockDim.x * 8;   // eight ids per thread are requested together
    for (int i0 = 0; i0 < n_slots; i0 += per_round) {
        int ev[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = i0 + j * (int)blockDim.x + (int)threadIdx.x;
            ev[j] = i < n_slots ? __ldg(expert_ids + i) : -1;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int e = ev[j];
            if (e < -1 || e >= E) { bad = true; e = -1; }
            const unsigned peers = __match_any_sync(0xffffffffu, e);
            if (e >= 0 && lane == __ffs(peers) - 1) atomicAdd(&s_cnt[e], __popc(peers));
        }
    }
    if (bad) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
    __syncthreads();
    if (threadIdx.x < 32) {   // exclusive prefix sums over the experts, 32 at a time
        int row0 = 0, tile0 = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int c = e < E ? s_cnt[e] : 0;
            const int t = (c + tile_rows - 1) / tile_rows;
            int ic = c, it = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int vc = __shfl_up_sync(0xffffffffu, ic, o), vt = __shfl_up_sync(0xffffffffu, it, o);
                if (lane >= o) { ic += vc; it += vt; }
            }
            if (e < E) {
                plan.list_row0[e] = row0 + ic - c;
                plan.tile_start[e] = tile0 + it - t;
                s_cur[e] = row0 + ic - c;
            }
            row0 += __shfl_sync(0xffffffffu, ic, 31);
            tile0 += __shfl_sync(0xffffffffu, it, 31);
        }
        if (lane == 0) { plan.list_row0[E] = row0; plan.tile_start[E] = tile0; }
    }
    __syncthreads();
    for (int i0 = 0; i0 < n_slots; i0 += per_round) {
        int ev[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = i0 + j * (int)blockDim.x + (int)threadIdx.x;
            ev[j] = i < n_slots ? __ldg(expert_ids + i) : -1;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = i0 + j * (int)blockDim.x + (int)threadIdx.x;
            int e = ev[j];
            if (e < -1 || e >= E) e = -1;
            const unsigned peers = __match_any_sync(0xffffffffu, e);
            const int leader = __ffs(peers) - 1;
            int base = 0;
            if (e >= 0 && lane == leader) base = atomicAdd(&s_cur[e], __popc(peers));
            const int pos = __shfl_sync(0xffffffffu, base, leader) + __popc(peers & ((1u << lane) - 1u));
            if (e >= 0) {
                plan.rowidx[pos] = i / top_k;   // row of X: the token
                plan.rowout[pos] = i;           // row of the staging buffer: (token, slot)
            }
        }
    }
}

template <typename T> struct Vec16;
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };
template <> struct Vec16<__half> { static constexpr int N = 8; };

__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint4 pack16(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
__device__ __forceinline__ uint4 pack16(const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<const uint32_t*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void unpack16_half(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        f[2 * i] = p.x;
        f[2 * i + 1] = p.y;
    }
}
__device__ __forceinline__ uint4 pack16_half(const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2 p = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<const uint32_t*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// y_t = sum_j weight[t][j] * staged[t*top_k + j]  over the routed slots, 16 bytes per thread.
template <typename T>
__global__ void __launch_bounds__(256)
moe_combine_kernel(const uint4* __restrict__ staged, const int32_t* __restrict__ expert_ids,
                   const float* __restrict__ weights, long long N, int vpr, int E, int top_k,
                   uint4* __restrict__ Y) {
    constexpr int NV = Vec16<T>::N;
    constexpr bool IS_BF16 = sizeof(T) == 2 && Vec16<T>::N == 8 && __is_same(T, __nv_bfloat16);
    const long long total = N * vpr;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long t = i / vpr;
        const int v = (int)(i % vpr);
        float acc[NV];
#pragma unroll
        for (int c = 0; c < NV; ++c) acc[c] = 0.f;
        // four slots at a time: ids, weights and staged rows are requested together (a staged row is
        // read whether or not its slot is routed -- the buffer is there -- and dropped afterwards, so
        // that the row does not wait for the id); the sum runs in slot order
        for (int j0 = 0; j0 < top_k; j0 += 4) {
            int e[4];
            float g[4];
            uint4 raw[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = j0 + u;
                e[u] = -1;
                if (j < top_k) {
                    e[u] = __ldg(expert_ids + t * top_k + j);
                    g[u] = __ldg(weights + t * top_k + j);
                    raw[u] = __ldg(&staged[(t * top_k + j) * vpr + v]);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (e[u] < 0 || e[u] >= E) continue;
                float f[NV];
                if constexpr (sizeof(T) == 2 && !IS_BF16) unpack16_half(raw[u], f);
                else unpack16(raw[u], f);
#pragma unroll
                for (int c = 0; c < NV; ++c) acc[c] = fmaf(g[u], f[c], acc[c]);
            }
        }
        if constexpr (sizeof(T) == 2 && !IS_BF16) Y[i] = pack16_half(acc);
        else Y[i] = pack16(acc);
    }
}

struct MoeWs {
    FfnPlan plan;
    int32_t *counts, *cursor;
    void* staged;
    void* packed;
    bool ok;
    size_t used;
};

sentry_ffn_desc as_ffn_desc(const sentry_moe_desc& m) {
    sentry_ffn_desc d;
    d.B = 1;
    d.T = 1;   // the row count of the plan is N * top_k; the fused-pair kernels read it from the plan
    d.D = m.D; d.F = m.F; d.k_c = m.k_c; d.n_lists = m.E; d.dtype = m.dtype;
    return d;
}

MoeWs carve(const sentry_moe_desc& m, void* ws, size_t bytes, bool with_weights) {
    WsAlloc a(ws, bytes);
    MoeWs w;
    const size_t slots = (size_t)m.N * m.top_k;
    const size_t esz = m.dtype == SENTRY_F32 ? 4 : 2;
    w.plan.sample_row0 = a.take<int32_t>(1);
    w.plan.list_row0 = a.take<int32_t>((size_t)m.E + 1);
    w.plan.tile_start = a.take<int32_t>((size_t)m.E + 1);
    w.plan.rowidx = a.take<int32_t>(slots);
    w.plan.rowout = a.take<int32_t>(slots);
    w.counts = a.take<int32_t>((size_t)2 * m.E);
    w.cursor = w.counts ? w.counts + m.E : nullptr;
    w.staged = a.take<uint8_t>(slots * m.D * esz);
    w.packed = with_weights ? a.take<uint8_t>(ffn_packed_bytes(as_ffn_desc(m))) : nullptr;
    w.ok = a.ok;
    w.used = a.off;
    return w;
}

}  // namespace

size_t moe_workspace_bytes(const sentry_moe_desc& m) { return carve(m, nullptr, 0, true).used + 256; }
size_t moe_packed_bytes(const sentry_moe_desc& m) { return ffn_packed_bytes(as_ffn_desc(m)); }

int launch_moe_prepack(sentry_ctx* ctx, const MoeArgs& m, void* packed, cudaStream_t st) {
    FfnArgs a = {};
    a.d = as_ffn_desc(m.d);
    a.W1 = m.W1; a.W2 = m.W2;
    a.kept = m.kept;
    a.w_stride = (size_t)m.d.D * m.d.F;
    a.status = m.status;
    return launch_ffn_prepack(ctx, a, packed, st);
}

int launch_moe_ffn(sentry_ctx* ctx, const MoeArgs& m, void* ws, size_t ws_bytes, const void* packed,
                   cudaStream_t st) {
    const sentry_moe_desc& d = m.d;
    MoeWs w = carve(d, ws, ws_bytes, packed == nullptr);
    if (!w.ok) return SENTRY_ERR_WORKSPACE;
    const sentry_ffn_desc fd = as_ffn_desc(d);
    const int tile_rows = ffn_tile_rows(fd);
    const long long slots = (long long)d.N * d.top_k;
    const unsigned route_blocks = (unsigned)((slots + kPlanThreads * 8 - 1) / (kPlanThreads * 8));
    const size_t route_smem = (size_t)2 * d.E * sizeof(int);

    if (packed == nullptr) {
        int rc = launch_moe_prepack(ctx, m, w.packed, st);
        if (rc != SENTRY_OK) return rc;
        packed = w.packed;
    }
    if (slots <= kPlanOneMaxSlots && route_smem <= 48 * 1024) {
        LaunchScope ls(ctx, KS_MOE_PLAN, st);
        moe_plan_one_kernel<<<1, kPlanOneThreads, route_smem, st>>>(m.expert_ids, (int)slots, d.E, d.top_k, tile_rows,
                                                                    w.plan, m.status);
    } else {
        SENTRY_CUDA_TRY(cudaMemsetAsync(w.counts, 0, (size_t)d.E * sizeof(int32_t), st));
        LaunchScope ls(ctx, KS_MOE_PLAN, st, 3);
        moe_route_kernel<<<route_blocks, kPlanThreads, route_smem, st>>>(m.expert_ids, slots, d.E, d.top_k, 0,
                                                                         w.counts, w.cursor, w.plan, m.status);
        moe_offsets_kernel<<<1, kPlanThreads, 0, st>>>(w.counts, d.E, tile_rows, w.plan, w.cursor);
        moe_route_kernel<<<route_blocks, kPlanThreads, route_smem, st>>>(m.expert_ids, slots, d.E, d.top_k, 1,
                                                                         w.counts, w.cursor, w.plan, m.status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());

    FfnArgs a = {};
    a.d = fd;
    a.X = m.X;
    a.Y = w.staged;
    a.status = m.status;
    const int kc_pad = ffn_kc_pad(fd);
    const int max_tiles = (int)((slots + tile_rows - 1) / tile_rows) + d.E;
    void* w1p = const_cast<void*>(packed);
    void* w2p = (uint8_t*)w1p + ffn_packed_bytes(fd) / 2;
    int rc = launch_ffn_main(ctx, a, w.plan, w1p, w2p, kc_pad, max_tiles, st);
    if (rc != SENTRY_OK) return rc;

    {
        const int esz = d.dtype == SENTRY_F32 ? 4 : 2;
        const int vpr = d.D * esz / 16;
        const long long total = (long long)d.N * vpr;
        long long blocks = (total + 255) / 256;
        const long long cap = (long long)ctx->sm_count * 16;
        if (blocks > cap) blocks = cap;
        LaunchScope ls(ctx, KS_MOE_COMBINE, st);
        if (d.dtype == SENTRY_F32)
            moe_combine_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(
                (const uint4*)w.staged, m.expert_ids, m.expert_weights, d.N, vpr, d.E, d.top_k, (uint4*)m.Y);
        else if (d.dtype == SENTRY_F16)
            moe_combine_kernel<__half><<<(unsigned)blocks, 256, 0, st>>>(
                (const uint4*)w.staged, m.expert_ids, m.expert_weights, d.N, vpr, d.E, d.top_k, (uint4*)m.Y);
        else
            moe_combine_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(
                (const uint4*)w.staged, m.expert_ids, m.expert_weights, d.N, vpr, d.E, d.top_k, (uint4*)m.Y);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

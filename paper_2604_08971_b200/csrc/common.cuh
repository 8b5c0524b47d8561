// Shared declarations of the sentry CUDA library: context, launch helpers and
// small device utilities used by several kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/sentry.h"

// Kernel slots for launch accounting and optional per-kernel timing.
enum KernelSlot {
    KS_GATE_ROWS = 0, KS_GATE_EXPAND, KS_ATT_SCORE, KS_ATT_SELECT, KS_ATT_CORE,
    KS_FFN_PREPARE, KS_FFN_MAIN, KS_GATE_EVAL, KS_PROJ_QKV, KS_PROJ_OUT,
    KS_MOE_PLAN, KS_MOE_COMBINE, KS_TABLE_ARRANGE, KS_COUNT
};

struct ProfRec { cudaEvent_t start, stop; int slot; };

struct sentry_ctx {
    int device;
    void* workspace;
    size_t workspace_bytes;
    unsigned int* d_status;  // device status word (SENTRY_STATUS_BIT_*)
    int last_launches;
    int sm_count;
    bool profiling;
    int attend_kernel;       // SENTRY_ATTEND_AUTO / _WARP_MMA / _TCGEN05
    int long_select;         // SENTRY_LONG_SELECT_AUTO / _QUERY_BLOCKS / _PER_GROUP
    std::vector<ProfRec> prof;      // events recorded since profiling was enabled
    std::vector<cudaEvent_t> pool;  // reusable events
};

// Brackets one kernel launch with events when profiling is on; counts the launch.
struct LaunchScope {
    sentry_ctx* ctx; cudaStream_t st; ProfRec rec; bool on;
    // `launches`: kernels the scope covers (they are timed together under `slot`)
    LaunchScope(sentry_ctx* c, int slot, cudaStream_t s, int launches = 1) : ctx(c), st(s), on(c->profiling) {
        ctx->last_launches += launches;
        if (!on) return;
        cudaEvent_t ev[2];
        for (int i = 0; i < 2; ++i) {
            if (!ctx->pool.empty()) { ev[i] = ctx->pool.back(); ctx->pool.pop_back(); }
            else if (cudaEventCreate(&ev[i]) != cudaSuccess) { on = false; return; }
        }
        rec.start = ev[0]; rec.stop = ev[1]; rec.slot = slot;
        cudaEventRecord(rec.start, st);
    }
    ~LaunchScope() {
        if (!on) return;
        cudaEventRecord(rec.stop, st);
        ctx->prof.push_back(rec);
    }
};

#define SENTRY_CUDA_TRY(expr)                         \
    do {                                              \
        cudaError_t _e = (expr);                      \
        if (_e != cudaSuccess) return SENTRY_ERR_CUDA; \
    } while (0)

// Makes `device` current for the lifetime of the object and puts the caller's device back
// afterwards, so that no entry point changes the calling thread's current device.
struct DeviceGuard {
    int prev;
    bool ok, switched;
    explicit DeviceGuard(int device) : prev(-1), ok(false), switched(false) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        if (prev != device) {
            if (cudaSetDevice(device) != cudaSuccess) return;
            switched = true;
        }
        ok = true;
    }
    ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
    DeviceGuard(const DeviceGuard&) = delete;
    DeviceGuard& operator=(const DeviceGuard&) = delete;
};
#define SENTRY_ON_DEVICE(device)      \
    DeviceGuard _dev_guard(device);   \
    if (!_dev_guard.ok) return SENTRY_ERR_CUDA

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Bump allocator over the caller-provided workspace.
struct WsAlloc {
    char* base;
    size_t cap, off;
    bool ok;
    WsAlloc(void* p, size_t bytes) : base((char*)p), cap(bytes), off(0), ok(true) {}
    template <typename T>
    T* take(size_t n) {
        size_t o = align_up(off, 256);
        size_t end = o + n * sizeof(T);
        if (end > cap || base == nullptr) { ok = false; off = end; return nullptr; }
        off = end;
        return (T*)(base + o);
    }
};

// ---- U = c * ceil(ln T_v), clamped to [1, T_v] (Section 4.4).  ceil(ln T) is
// the smallest k with T <= floor(e^k); the thresholds are integers so host and
// device agree exactly.
__host__ __device__ inline int sentry_ceil_ln(int T) {
    const unsigned int fl_exp[22] = {1u, 2u, 7u, 20u, 54u, 148u, 403u, 1096u, 2980u, 8103u,
                                     22026u, 59874u, 162754u, 442413u, 1202604u, 3269017u,
                                     8886110u, 24154952u, 65659969u, 178482300u, 485165195u,
                                     1318815734u};
    int k = 0;
    while (k < 21 && (unsigned int)T > fl_exp[k]) ++k;
    if ((unsigned int)T > fl_exp[21]) k = 22;
    return k;
}
__host__ __device__ inline int sentry_num_active(int T_v, int c) {
    if (T_v <= 0) return 0;
    long long u = (long long)c * sentry_ceil_ln(T_v);
    if (u > T_v) u = T_v;
    if (u < 1) u = 1;
    return (int)u;
}

#ifdef __CUDACC__
// Order-preserving map float -> uint32 for "score descending" selection:
// larger score -> larger key; +0 and -0 map to the same key; NaN -> 0 (below -inf).
__device__ __forceinline__ uint32_t sentry_order_key(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Block-wide sum of an int (all threads get the result).  `red` = 33 ints of smem.
__device__ __forceinline__ int block_sum_int(int v, int* red) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();  // protect `red` from the previous use
    if (lane == 0) red[wid] = v;
    __syncthreads();
    int t = 0;
    for (int w = 0; w < nw; ++w) t += red[w];
    return t;
}

// Top-k of n keys by rank counting, for rows short enough that n^2 comparisons are cheaper
// than 32 rounds of block-wide counting: element i is kept iff fewer than k elements come
// before it in the order (larger key first, equal keys -> lower index first).  Same contract
// as block_select_topk.
__device__ inline void block_select_topk_rank(const uint32_t* keys, int n, int k, int32_t* out,
                                              const uint16_t* remap, int* red) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    int* wk = red;
    int base = 0;
    for (int i0 = 0; i0 < n; i0 += blockDim.x) {
        const int i = i0 + threadIdx.x;
        bool keep = false;
        if (i < n) {
            const uint32_t mine = keys[i];
            int before = 0;
            for (int j = 0; j < i; ++j) before += (keys[j] >= mine);      // earlier index wins ties
            for (int j = i + 1; j < n; ++j) before += (keys[j] > mine);
            keep = before < k;
        }
        const unsigned km = __ballot_sync(0xffffffffu, keep);
        __syncthreads();
        if (lane == 0) wk[wid] = __popc(km);
        __syncthreads();
        int pos = base, tot = 0;
        for (int w = 0; w < nw; ++w) { if (w < wid) pos += wk[w]; tot += wk[w]; }
        if (keep) out[pos + __popc(km & ((1u << lane) - 1u))] = remap ? (int32_t)remap[i] : i;
        base += tot;
    }
    __syncthreads();
}

// Top-k of n keys held in shared memory, larger key first, equal keys -> lower
// index first.  Writes the selected indices to out[0..k) in ASCENDING index
// order, mapped through `remap` (uint16 list) when given.  All threads of the
// block must call it.  `red` = 33 ints of smem.  Requires 1 <= k <= n.
__device__ inline void block_select_topk(const uint32_t* keys, int n, int k, int32_t* out,
                                         const uint16_t* remap, int* red) {
    if (n <= 256) { block_select_topk_rank(keys, n, k, out, remap, red); return; }
    // 1. t = the k-th largest key, by radix selection: four passes over 8-bit digits, each a
    //    shared-memory histogram of the keys that still match the digits fixed so far, scanned
    //    from the top digit down by one warp.
    __shared__ int s_hist[256];
    __shared__ int s_pick[2];   // chosen digit, keys still to take inside it
    uint32_t prefix = 0, fixed = 0;
    int want = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) s_hist[i] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const uint32_t key = keys[i];
            if ((key & fixed) == prefix) atomicAdd(&s_hist[(key >> shift) & 255u], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane L owns digits 255-8L .. 248-8L (descending); inclusive scan over lanes
            const int top = 255 - 8 * (int)threadIdx.x;
            int mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += s_hist[top - j];
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if ((int)threadIdx.x >= o) incl += v;
            }
            const int above = incl - mine;               // keys in digits above this lane's
            if (above < want && want <= incl) {          // the k-th key falls into this lane's digits
                int acc = above;
                for (int j = 0; j < 8; ++j) {
                    const int c = s_hist[top - j];
                    if (want <= acc + c) { s_pick[0] = top - j; s_pick[1] = want - acc; break; }
                    acc += c;
                }
            }
        }
        __syncthreads();
        prefix |= (uint32_t)s_pick[0] << shift;
        fixed |= 255u << shift;
        want = s_pick[1];
    }
    const uint32_t t = prefix;
    const int gt = k - want;     // keys strictly above t; `want` of the keys equal to t are taken
    const int need_eq = k - gt;
    // 2. ordered compaction: everything above t, plus the first need_eq equal to t
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    int base = 0, eq_seen = 0;
    int* wk = red;            // [nw] keep counts
    int* we = red + 33;       // [nw] eq counts  (caller provides 66 ints in total)
    for (int i0 = 0; i0 < n; i0 += blockDim.x) {
        const int i = i0 + threadIdx.x;
        const bool in = i < n;
        const uint32_t key = in ? keys[i] : 0u;
        const bool is_eq = in && key == t;
        const bool is_gt = in && key > t;
        const unsigned em = __ballot_sync(0xffffffffu, is_eq);
        __syncthreads();
        if (lane == 0) we[wid] = __popc(em);
        __syncthreads();
        int eq_before = eq_seen;
        for (int w = 0; w < wid; ++w) eq_before += we[w];
        int eq_total = 0;
        for (int w = 0; w < nw; ++w) eq_total += we[w];
        const int eq_rank = eq_before + __popc(em & ((1u << lane) - 1u));
        const bool keep = is_gt || (is_eq && eq_rank < need_eq);
        const unsigned km = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) wk[wid] = __popc(km);
        __syncthreads();
        int pos = base;
        for (int w = 0; w < wid; ++w) pos += wk[w];
        int k_total = 0;
        for (int w = 0; w < nw; ++w) k_total += wk[w];
        if (keep) out[pos + __popc(km & ((1u << lane) - 1u))] = remap ? (int32_t)remap[i] : i;
        base += k_total;
        eq_seen += eq_total;
    }
    __syncthreads();
}

// Present-token list of one sample: valid[p] = p-th token t (ascending) whose
// modality bit ids[t] is set in `mask`.  Returns T_v to every thread.  ids ==
// nullptr means every token is present.  `red` = 66 ints of smem.
__device__ inline int block_build_valid(const int32_t* ids, int T, uint32_t mask,
                                        uint16_t* valid, int* red) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    int base = 0;
    for (int t0 = 0; t0 < T; t0 += blockDim.x) {
        const int t = t0 + threadIdx.x;
        bool ok = false;
        if (t < T) {
            if (ids == nullptr) ok = true;
            else {
                const int m = ids[t];
                ok = (m >= 0 && m < 32) && ((mask >> m) & 1u);
            }
        }
        const unsigned bm = __ballot_sync(0xffffffffu, ok);
        __syncthreads();
        if (lane == 0) red[wid] = __popc(bm);
        __syncthreads();
        int pos = base, tot = 0;
        for (int w = 0; w < nw; ++w) { if (w < wid) pos += red[w]; tot += red[w]; }
        if (ok) valid[pos + __popc(bm & ((1u << lane) - 1u))] = (uint16_t)t;
        base += tot;
    }
    __syncthreads();
    return base;
}

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <> __device__ __forceinline__ float to_f32<__half>(__half x) { return __half2float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }
template <> __device__ __forceinline__ __half from_f32<__half>(float x) { return __float2half_rn(x); }
template <> __device__ __forceinline__ uint8_t from_f32<uint8_t>(float) { return 0; }   // only the zero of the FP8 weight gather
#endif  // __CUDACC__

// ---- launchers implemented in the .cu files (host side; return sentry_status)
int launch_gate_select_multi(sentry_ctx* ctx, int S, const sentry_gate_set* sets, int n_sets, int32_t* const* ws_rows,
                             uint32_t* const* ws_groups, cudaStream_t st);
int launch_gate_select(sentry_ctx* ctx, const float* scores, int S, int n_units,
                       const uint32_t* masks, int n_masks, int k, int32_t* kept,
                       uint32_t* kv_groups, int heads_per_group, int32_t* ws_rows,
                       uint32_t* ws_groups, cudaStream_t st);

int launch_gate_eval(sentry_ctx* ctx, const float* zeta, const float* gamma, const int32_t* layer_offsets,
                     int n_layers, const float* W1, const float* b1, const float* w2, const float* b2, int M,
                     int hidden, int N, float* logits, float* gates, cudaStream_t st);
int launch_layer_counts(sentry_ctx* ctx, const int32_t* kept, int n_masks, int k, const int32_t* layer_offsets,
                        int n_layers, int32_t* counts, cudaStream_t st);

struct AttendArgs {
    sentry_attend_desc d;
    const void *Q, *K, *V;
    const int32_t* kept_heads;
    const int32_t* ids;
    const uint32_t* masks;
    const int32_t* sample_table;
    const int64_t* sample_offsets;
    int n_subsets;
    void* O;
    int32_t* active;        // [B,k_h,U_max] written by selection or given by the caller
    int32_t* active_out_user;  // the caller's active_out (may be null)
    bool selection_given;   // true: `active` is the caller's forced selection
    float* mscore;          // workspace [B,k_h,T]
    int U_max;
    unsigned int* status;
    // head selection inside the attention launch (null: kept_heads is given)
    const float* gate_scores;   // [gate_S, Hq] score table of the heads
    int gate_S;
    int32_t* kept_out;          // [B,k_h] where the kernel leaves the lists it selected
};
int launch_attend_generic(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st);
bool attend_tc_supported(const sentry_attend_desc& d);
int launch_table_arrange(sentry_ctx* ctx, const int32_t* ids, int T, int c, const int32_t* table,
                         const int64_t* offsets, int n_subsets, int32_t* out, cudaStream_t st);
bool attend_long_select_supported(const sentry_attend_desc& d);
int launch_attend_long_select(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st);
int launch_attend_tc(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st);
bool attend_bf16_supported(const sentry_attend_desc& d);
bool attend_bf16_gate_fusable(const sentry_attend_desc& d);
int launch_attend_bf16(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st);
// the same kernels compiled for IEEE-half tensors (attend_f16.cu, attend_long_f16.cu)
bool attend_long_select_f16_supported(const sentry_attend_desc& d);
int launch_attend_long_select_f16(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st);
bool attend_f16_supported(const sentry_attend_desc& d);
bool attend_f16_gate_fusable(const sentry_attend_desc& d);
int launch_attend_f16(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st);

struct ProjArgs {
    sentry_proj_desc d;
    const void *X, *WQ, *WK, *WV;     // QKV projection
    const void *A, *WO;               // output projection
    const int32_t* kept_heads;
    const int32_t* ids;
    const uint32_t* masks;
    void *Q, *K, *V, *out;
    unsigned int* status;
};
int launch_project_qkv_generic(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st);
int launch_project_out_generic(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st);
bool project_qkv_tc_supported(const sentry_proj_desc& d);
bool project_out_tc_supported(const sentry_proj_desc& d);
int launch_project_qkv_tc(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st);
int launch_project_out_tc(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st);
bool project_qkv_tc_f16_supported(const sentry_proj_desc& d);   // the same for IEEE-half tensors (proj_tc_f16.cu)
bool project_out_tc_f16_supported(const sentry_proj_desc& d);
int launch_project_qkv_tc_f16(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st);
int launch_project_out_tc_f16(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st);

struct FfnArgs {
    sentry_ffn_desc d;
    const void *X, *W1, *W2;
    const int32_t* kept;
    size_t w_stride;        // elements between the weight matrices of consecutive lists (0: shared)
    float fp8_a_scale, fp8_h_inv, fp8_y_scale;   // FP8 form: scale of GEMM1's accumulator, 1 / hidden scale, scale of Y
    const int32_t* list_of_sample;
    const int32_t* ids;
    const uint32_t* masks;
    void* Y;
    unsigned int* status;
};
size_t ffn_workspace_bytes(const sentry_ffn_desc& d);
size_t ffn_packed_bytes(const sentry_ffn_desc& d);
bool ffn_tc_fp8_supported(const sentry_ffn_desc& d);
int launch_ffn_prepack(sentry_ctx* ctx, const FfnArgs& a, void* packed, cudaStream_t st);
int launch_ffn_prepack_fp8(sentry_ctx* ctx, const sentry_ffn_desc& d, const uint8_t* W1q, const uint8_t* W2q, float s1,
                           float s2, const int32_t* kept, void* packed, cudaStream_t st);
int launch_wait_expiry_selftest(sentry_ctx* ctx, long long limit_cycles, cudaStream_t st);
int launch_ffn(sentry_ctx* ctx, const FfnArgs& a, void* ws, size_t ws_bytes, const void* packed, cudaStream_t st);
int ffn_kc_pad(const sentry_ffn_desc& d);
int ffn_tile_rows(const sentry_ffn_desc& d);

struct MoeArgs {
    sentry_moe_desc d;
    const void *X, *W1, *W2;
    const int32_t* kept;            // [E, k_c]
    const int32_t* expert_ids;      // [N, top_k]
    const float* expert_weights;    // [N, top_k]
    void* Y;
    unsigned int* status;
};
size_t moe_workspace_bytes(const sentry_moe_desc& m);
size_t moe_packed_bytes(const sentry_moe_desc& m);
int launch_moe_prepack(sentry_ctx* ctx, const MoeArgs& m, void* packed, cudaStream_t st);
int launch_moe_ffn(sentry_ctx* ctx, const MoeArgs& m, void* ws, size_t ws_bytes, const void* packed, cudaStream_t st);

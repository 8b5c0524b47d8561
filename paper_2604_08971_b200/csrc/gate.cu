// SentryGate selection (Section 4.6): per modality-mask row of the score
// table, keep the k best-scoring units; then fan the per-row result out to the
// per-sample masks.  Selection is exact and deterministic: scores are mapped to
// order-preserving integer keys, the k-th key is found by a bitwise threshold
// search with warp-ballot counting, and the kept indices are compacted in
// ascending order (equal scores: lower index first).
#include "common.cuh"

namespace {

constexpr int kGateMaxThreads = 1024;

// Block size of the per-row selection: one key per thread up to 1024 threads.
inline int gate_threads(int n_units) {
    int t = (n_units + 31) / 32 * 32;
    return t < 64 ? 64 : (t > kGateMaxThreads ? kGateMaxThreads : t);
}

// One block per score-table row s: rows[s, 0..k) and groups[s].  With fan_masks given (a small
// fan-out), the block also copies its row to every sample whose mask selects it, which saves
// the second launch: kept[m, :] = rows[s, :] for masks[m] == s.
__device__ __forceinline__ void
gate_row_block(int s, const float* __restrict__ scores, int n_units, int k,
               int32_t* __restrict__ rows, uint32_t* __restrict__ groups,
               int heads_per_group, const uint32_t* __restrict__ fan_masks,
               int n_masks, int S, int32_t* __restrict__ kept,
               uint32_t* __restrict__ kv_groups, unsigned int* status) {
    extern __shared__ uint32_t s_keys[];
    __shared__ int red[66];
    __shared__ uint32_t s_bits;
    const float* row = scores + (size_t)s * n_units;
    for (int i = threadIdx.x; i < n_units; i += blockDim.x) s_keys[i] = sentry_order_key(row[i]);
    if (threadIdx.x == 0) s_bits = 0u;
    __syncthreads();
    int32_t* out = rows + (size_t)s * k;
    block_select_topk(s_keys, n_units, k, out, nullptr, red);
    if (groups != nullptr) {
        uint32_t bits = 0u;
        for (int i = threadIdx.x; i < k; i += blockDim.x) bits |= 1u << (out[i] / heads_per_group);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
        if ((threadIdx.x & 31) == 0 && bits) atomicOr(&s_bits, bits);
        __syncthreads();
        if (threadIdx.x == 0) groups[s] = s_bits;
    }
    if (fan_masks == nullptr) return;
    __syncthreads();   // out[] (global, written by this block) is complete
    if (k <= 32) {
        // short lists (heads): one thread per mask -- one independent load of the mask per
        // thread instead of a chain of dependent loads down an element loop
        for (int m = threadIdx.x; m < n_masks; m += blockDim.x) {
            const uint32_t ms = fan_masks[m];
            if (ms == (uint32_t)s) {
                int32_t* dst = kept + (size_t)m * k;
                for (int j = 0; j < k; ++j) dst[j] = out[j];
                if (kv_groups != nullptr) kv_groups[m] = s_bits;
            } else if (s == 0 && ms >= (uint32_t)S) {
                atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            }
        }
        return;
    }
    const long long total = (long long)n_masks * k;
    for (long long i = threadIdx.x; i < total; i += blockDim.x) {
        const int m = (int)(i / k), j = (int)(i % k);
        const uint32_t ms = fan_masks[m];
        if (ms == (uint32_t)s) {
            kept[i] = out[j];
            if (j == 0 && kv_groups != nullptr) kv_groups[m] = s_bits;
        } else if (s == 0 && j == 0 && ms >= (uint32_t)S) {
            atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
        }
    }
}

__global__ void __launch_bounds__(kGateMaxThreads)
gate_rows_kernel(const float* __restrict__ scores, int n_units, int k,
                 int32_t* __restrict__ rows, uint32_t* __restrict__ groups,
                 int heads_per_group, const uint32_t* __restrict__ fan_masks = nullptr,
                 int n_masks = 0, int S = 0, int32_t* __restrict__ kept = nullptr,
                 uint32_t* __restrict__ kv_groups = nullptr, unsigned int* status = nullptr) {
    gate_row_block(blockIdx.x, scores, n_units, k, rows, groups, heads_per_group, fan_masks, n_masks, S, kept,
                   kv_groups, status);
}

// Several selections over the same S mask values (heads and channels of a layer, or several
// layers) in one launch: block b works on row b % S of set b / S.
struct GateSetDev {
    const float* scores;
    int n_units, k;
    int32_t* rows;
    uint32_t* groups;
    int heads_per_group;
    const uint32_t* fan_masks;   // null: no fan-out in this launch (the set is expanded afterwards)
    int n_masks;
    int32_t* kept;
    uint32_t* kv_groups;
};
struct GateSetsDev { GateSetDev set[SENTRY_GATE_MAX_SETS]; };

__global__ void __launch_bounds__(kGateMaxThreads)
gate_rows_multi_kernel(const __grid_constant__ GateSetsDev sets, int S, unsigned int* status) {
    const GateSetDev& g = sets.set[blockIdx.x / S];
    gate_row_block((int)(blockIdx.x % S), g.scores, g.n_units, g.k, g.rows, g.groups, g.heads_per_group,
                   g.fan_masks, g.n_masks, S, g.kept, g.kv_groups, status);
}

// kept[m, :] = rows[masks[m], :]  (and kv_groups[m] = groups[masks[m]]).
__global__ void gate_expand_kernel(const int32_t* __restrict__ rows,
                                   const uint32_t* __restrict__ groups,
                                   const uint32_t* __restrict__ masks, int S, int n_masks, int k,
                                   int32_t* __restrict__ kept, uint32_t* __restrict__ kv_groups,
                                   unsigned int* status) {
    const size_t total = (size_t)n_masks * k;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / k), j = (int)(i % k);
        const uint32_t s = masks[m];
        if (s >= (uint32_t)S) {
            if (j == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            continue;
        }
        kept[i] = rows[(size_t)s * k + j];
        if (j == 0 && kv_groups != nullptr) kv_groups[m] = groups[s];
    }
}

}  // namespace

int launch_gate_select(sentry_ctx* ctx, const float* scores, int S, int n_units,
                       const uint32_t* masks, int n_masks, int k, int32_t* kept,
                       uint32_t* kv_groups, int heads_per_group, int32_t* ws_rows,
                       uint32_t* ws_groups, cudaStream_t st) {
    const size_t smem = (size_t)n_units * sizeof(uint32_t);
    if (smem > 48 * 1024)
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(gate_rows_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const size_t total = (size_t)n_masks * k;
    if (total <= 16384) {   // small fan-out: one launch does both steps
        // enough threads for the fan-out as well as for the selection
        int threads = gate_threads(n_units);
        const int fan = k <= 32 ? n_masks : (int)(total < 1024 ? total : 1024);
        while (threads < 256 && threads < fan) threads *= 2;
        LaunchScope ls(ctx, KS_GATE_ROWS, st);
        gate_rows_kernel<<<S, threads, smem, st>>>(
            scores, n_units, k, ws_rows, kv_groups ? ws_groups : nullptr,
            heads_per_group > 0 ? heads_per_group : 1, masks, n_masks, S, kept, kv_groups, ctx->d_status);
        SENTRY_CUDA_TRY(cudaGetLastError());
        return SENTRY_OK;
    }
    {
        LaunchScope ls(ctx, KS_GATE_ROWS, st);
        gate_rows_kernel<<<S, gate_threads(n_units), smem, st>>>(scores, n_units, k, ws_rows,
                                                         kv_groups ? ws_groups : nullptr,
                                                         heads_per_group > 0 ? heads_per_group : 1);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    int blocks = (int)((total + 255) / 256);
    const int cap = ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    {
        LaunchScope ls(ctx, KS_GATE_EXPAND, st);
        gate_expand_kernel<<<blocks, 256, 0, st>>>(ws_rows, ws_groups, masks, S, n_masks, k, kept,
                                                   kv_groups, ctx->d_status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

// All sets in one launch; a set whose fan-out is large gets its rows there and one expand launch.
int launch_gate_select_multi(sentry_ctx* ctx, int S, const sentry_gate_set* sets, int n_sets, int32_t* const* ws_rows,
                             uint32_t* const* ws_groups, cudaStream_t st) {
    GateSetsDev dev = {};
    size_t smem = 0;
    int threads = 64;
    bool expand[SENTRY_GATE_MAX_SETS] = {};
    for (int i = 0; i < n_sets; ++i) {
        const sentry_gate_set& g = sets[i];
        const size_t total = (size_t)g.n_masks * g.k;
        expand[i] = total > 16384;
        GateSetDev& d = dev.set[i];
        d.scores = g.scores; d.n_units = g.n_units; d.k = g.k;
        d.rows = ws_rows[i];
        d.groups = g.kv_groups ? ws_groups[i] : nullptr;
        d.heads_per_group = g.heads_per_group > 0 ? g.heads_per_group : 1;
        d.fan_masks = expand[i] ? nullptr : g.masks;
        d.n_masks = g.n_masks; d.kept = g.kept; d.kv_groups = g.kv_groups;
        if ((size_t)g.n_units * sizeof(uint32_t) > smem) smem = (size_t)g.n_units * sizeof(uint32_t);
        int t = gate_threads(g.n_units);
        if (!expand[i]) {
            const int fan = g.k <= 32 ? g.n_masks : (int)(total < 1024 ? total : 1024);
            while (t < 256 && t < fan) t *= 2;
        }
        if (t > threads) threads = t;
    }
    if (smem > 48 * 1024)
        SENTRY_CUDA_TRY(cudaFuncSetAttribute(gate_rows_multi_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem));
    {
        LaunchScope ls(ctx, KS_GATE_ROWS, st);
        gate_rows_multi_kernel<<<S * n_sets, threads, smem, st>>>(dev, S, ctx->d_status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    for (int i = 0; i < n_sets; ++i) {
        if (!expand[i]) continue;
        const sentry_gate_set& g = sets[i];
        const size_t total = (size_t)g.n_masks * g.k;
        int blocks = (int)((total + 255) / 256);
        const int cap = ctx->sm_count * 8;
        if (blocks > cap) blocks = cap;
        LaunchScope ls(ctx, KS_GATE_EXPAND, st);
        gate_expand_kernel<<<blocks, 256, 0, st>>>(ws_rows[i], ws_groups[i], g.masks, S, g.n_masks, g.k, g.kept,
                                                   g.kv_groups, ctx->d_status);
        SENTRY_CUDA_TRY(cudaGetLastError());
    }
    return SENTRY_OK;
}

// ------------------------------------------------------------------------------------------
// Allocation-free variant of the gate selection.
//
// Its scratch (the per-score-row result that the fan-out kernel reads, the per-row KV-group
// bitmaps and a status word) lives in one file-scope device array instead of a workspace, so
// a caller that is not allowed to call cudaMalloc -- code running inside another runtime's
// memory pool, or an embedding that fixes its device-memory budget at start-up -- can still
// run the selection.  The array is part of the library image: every GPU that loads the
// library holds these 256 KB until the process exits.
//
// In host code `g_gate_scratch` is only a handle for the symbol, not a device address;
// the address a kernel can use comes from cudaGetSymbolAddress, asked once per device with
// that device current (static_scratch_of below).
#include <mutex>

namespace {

static __device__ __align__(256) unsigned char g_gate_scratch[SENTRY_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr size_t kStaticHeader = 256;  // status word, padded so the tables stay 256-byte aligned

struct StaticDevice {
    unsigned char* scratch = nullptr;  // device address of g_gate_scratch on this device
    int sm_count = 0;
};
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mu;

// Device address of the scratch array on `device` (which must be current).  The first call per
// device asks the runtime for it; later calls only read the cached value.
int static_scratch_of(int device, StaticDevice* out) {
    std::lock_guard<std::mutex> lock(g_static_mu);
    StaticDevice& sd = g_static_dev[device];
    if (sd.scratch == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_gate_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return SENTRY_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1)
            return SENTRY_ERR_CUDA;
        sd.sm_count = sms;
        sd.scratch = static_cast<unsigned char*>(p);
    }
    *out = sd;
    return SENTRY_OK;
}

}  // namespace

extern "C" int sentry_gate_select_static(int device, const float* scores, int S, int n_units,
                                         const uint32_t* masks, int n_masks, int k, int32_t* kept,
                                         uint32_t* kv_groups, int heads_per_group,
                                         uint32_t* status, void* stream) {
    if (scores == nullptr || masks == nullptr || kept == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (((uintptr_t)scores | (uintptr_t)masks | (uintptr_t)kept | (uintptr_t)kv_groups |
         (uintptr_t)status) % 4 != 0)
        return SENTRY_ERR_INVALID_ARG;
    if (device < 0 || device >= kMaxDevices) return SENTRY_ERR_INVALID_ARG;
    if (S < 1 || n_units < 1 || n_masks < 0 || k < 1 || k > n_units) return SENTRY_ERR_BAD_SHAPE;
    if (kv_groups != nullptr) {
        if (heads_per_group < 1) return SENTRY_ERR_INVALID_ARG;
        if ((n_units + heads_per_group - 1) / heads_per_group > 32) return SENTRY_ERR_BAD_SHAPE;
    }
    // the sort keys of one score row must fit the default shared-memory window
    if ((size_t)n_units * sizeof(uint32_t) > 48 * 1024) return SENTRY_ERR_UNSUPPORTED;
    // rows [S,k] i32 and groups [S] u32 must fit the static array
    const size_t rows_bytes = align_up((size_t)S * k * sizeof(int32_t), 256);
    const size_t groups_bytes = (size_t)S * sizeof(uint32_t);
    if (kStaticHeader + rows_bytes + groups_bytes > (size_t)SENTRY_STATIC_SCRATCH_BYTES)
        return SENTRY_ERR_WORKSPACE;
    if (n_masks == 0) return SENTRY_OK;

    SENTRY_ON_DEVICE(device);
    StaticDevice sd;
    int rc = static_scratch_of(device, &sd);
    if (rc != SENTRY_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned int* own_status = reinterpret_cast<unsigned int*>(sd.scratch);
    int32_t* rows = reinterpret_cast<int32_t*>(sd.scratch + kStaticHeader);
    uint32_t* groups = reinterpret_cast<uint32_t*>(sd.scratch + kStaticHeader + rows_bytes);
    // The array keeps whatever the previous call left.  rows/groups are rewritten in full for
    // all S score rows before the fan-out reads them; only the status word must start at zero.
    SENTRY_CUDA_TRY(cudaMemsetAsync(own_status, 0, sizeof(unsigned int), st));
    gate_rows_kernel<<<S, gate_threads(n_units), (size_t)n_units * sizeof(uint32_t), st>>>(
        scores, n_units, k, rows, kv_groups ? groups : nullptr, heads_per_group > 0 ? heads_per_group : 1);
    SENTRY_CUDA_TRY(cudaGetLastError());
    const size_t total = (size_t)n_masks * k;
    int blocks = (int)((total + 255) / 256);
    if (blocks > sd.sm_count * 8) blocks = sd.sm_count * 8;
    if (blocks < 1) blocks = 1;
    gate_expand_kernel<<<blocks, 256, 0, st>>>(rows, groups, masks, S, n_masks, k, kept, kv_groups,
                                               status != nullptr ? status : own_status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

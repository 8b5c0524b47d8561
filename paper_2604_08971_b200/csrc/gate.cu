// SentryGate selection (Section 4.6): per modality-mask row of the score
// table, keep the k best-scoring units; then fan the per-row result out to the
// per-sample masks.  Selection is exact and deterministic: scores are mapped to
// order-preserving integer keys, the k-th key is found by a bitwise threshold
// search with warp-ballot counting, and the kept indices are compacted in
// ascending order (equal scores: lower index first).
#include "common.cuh"

namespace {

constexpr int kGateThreads = 128;

// One block per score-table row s: rows[s, 0..k) and groups[s].
__global__ void __launch_bounds__(kGateThreads)
gate_rows_kernel(const float* __restrict__ scores, int n_units, int k,
                 int32_t* __restrict__ rows, uint32_t* __restrict__ groups,
                 int heads_per_group) {
    extern __shared__ uint32_t s_keys[];
    __shared__ int red[66];
    __shared__ uint32_t s_bits;
    const int s = blockIdx.x;
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
    {
        LaunchScope ls(ctx, KS_GATE_ROWS, st);
        gate_rows_kernel<<<S, kGateThreads, smem, st>>>(scores, n_units, k, ws_rows,
                                                         kv_groups ? ws_groups : nullptr,
                                                         heads_per_group > 0 ? heads_per_group : 1);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    const size_t total = (size_t)n_masks * k;
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

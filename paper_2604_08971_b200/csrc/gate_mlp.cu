// SentryGate evaluated on the device (Section 4.2, Eq. 1): for every unit i (attention head or FFN
// channel, the units of all layers concatenated) and every modality mask value s,
//   z_i(s) = zeta_i + gamma_l(i) * f_i(m_s),   g_i(s) = sigmoid(z_i(s)),
//   f_i(m) = w2_i . relu(W1_i m + b1_i) + b2_i        (a two-layer perceptron per unit),
// m_s = the bits of s.  The table of logits z [S, N] is what sentry_gate_select ranks: one row per
// mask value, so the "global threshold over all layers" of Section 4.6 is a top-k over the whole
// concatenated row; layer_counts then says how many of the kept units fall into each layer.
#include "common.cuh"

namespace {

// one thread per (mask value, unit); the few multiply-adds run in fp32 in the order of the definition
__global__ void __launch_bounds__(256)
gate_eval_kernel(const float* __restrict__ zeta, const float* __restrict__ gamma,
                 const int32_t* __restrict__ layer_offsets, int n_layers, const float* __restrict__ W1,
                 const float* __restrict__ b1, const float* __restrict__ w2, const float* __restrict__ b2,
                 int M, int hidden, int N, int S, float* __restrict__ logits, float* __restrict__ gates) {
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)S * N) return;
    const int s = (int)(idx / N), i = (int)(idx % N);
    int l = 0;
    while (l + 1 < n_layers && i >= layer_offsets[l + 1]) ++l;
    const float* W = W1 + (size_t)i * hidden * M;
    float f = b2[i];
    for (int j = 0; j < hidden; ++j) {
        float a = b1[(size_t)i * hidden + j];
        for (int q = 0; q < M; ++q)
            if ((s >> q) & 1) a += W[(size_t)j * M + q];
        f = fmaf(w2[(size_t)i * hidden + j], fmaxf(a, 0.f), f);
    }
    const float z = fmaf(gamma[l], f, zeta[i]);
    logits[idx] = z;
    if (gates != nullptr) gates[idx] = 1.0f / (1.0f + expf(-z));
}

// kept [n_masks, k] ascending unit indices -> counts [n_masks, n_layers]
__global__ void __launch_bounds__(256)
layer_count_kernel(const int32_t* __restrict__ kept, int n_masks, int k, const int32_t* __restrict__ layer_offsets,
                   int n_layers, int32_t* __restrict__ counts) {
    const int m = blockIdx.x;
    for (int l = threadIdx.x; l < n_layers; l += blockDim.x) {
        // kept is ascending: count = (first position >= end) - (first position >= begin)
        const int32_t* row = kept + (size_t)m * k;
        int pos[2];
        for (int e = 0; e < 2; ++e) {
            const int bound = layer_offsets[l + e];
            int lo = 0, hi = k;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (row[mid] < bound) lo = mid + 1; else hi = mid; }
            pos[e] = lo;
        }
        counts[(size_t)m * n_layers + l] = pos[1] - pos[0];
    }
}

}  // namespace

int launch_gate_eval(sentry_ctx* ctx, const float* zeta, const float* gamma, const int32_t* layer_offsets,
                     int n_layers, const float* W1, const float* b1, const float* w2, const float* b2, int M,
                     int hidden, int N, float* logits, float* gates, cudaStream_t st) {
    const int S = 1 << M;
    const size_t total = (size_t)S * N;
    LaunchScope ls(ctx, KS_GATE_EVAL, st);
    gate_eval_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(zeta, gamma, layer_offsets, n_layers, W1, b1, w2,
                                                                      b2, M, hidden, N, S, logits, gates);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

int launch_layer_counts(sentry_ctx* ctx, const int32_t* kept, int n_masks, int k, const int32_t* layer_offsets,
                        int n_layers, int32_t* counts, cudaStream_t st) {
    LaunchScope ls(ctx, KS_GATE_EVAL, st);
    layer_count_kernel<<<n_masks, 256, 0, st>>>(kept, n_masks, k, layer_offsets, n_layers, counts);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

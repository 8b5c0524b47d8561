// Projections of the pruned layer (Section 4.6, "Head pruning with GQA consistency"): only the
// column blocks of W_Q that belong to the kept heads, only the blocks of W_K / W_V of the KV groups
// those heads reference, only the row blocks of W_O of the kept heads, and only present tokens.
//   Q[b,h,t,:] = x_t . W_Q[:, h d:(h+1) d]  (h kept)      K, V[b,g,t,:] likewise (g referenced)
//   out[b,t,:] = sum_j A[b,j,t,:] . W_O[h_j d:(h_j+1) d, :]
// This file: the plain-ALU form (any dtype, fp32 accumulation), one CTA per token.
#include "common.cuh"

namespace {

constexpr int kProjThreads = 256;
constexpr int kMaxSlices = 96;   // kept heads + 2 x referenced groups

template <typename T>
__global__ void __launch_bounds__(kProjThreads)
project_qkv_kernel(const T* __restrict__ X, const T* __restrict__ WQ, const T* __restrict__ WK,
                   const T* __restrict__ WV, const int32_t* __restrict__ kept_heads,
                   const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks, int Tlen, int D, int Hq,
                   int Hk, int d, int k_h, T* __restrict__ Q, T* __restrict__ K, T* __restrict__ V,
                   unsigned int* status) {
    extern __shared__ float s_x[];                 // [D]
    __shared__ int s_kind[kMaxSlices], s_idx[kMaxSlices], s_n;
    const int b = blockIdx.x / Tlen, t = blockIdx.x % Tlen;
    const int m = ids[t];
    if (m < 0 || m >= 32 || !((masks[b] >> m) & 1u)) return;       // absent token: nothing is written
    if (threadIdx.x == 0) {
        // slices: one per kept head (Q), one K and one V per referenced group
        const int r = Hq / Hk;
        int n = 0;
        uint32_t groups = 0;
        for (int j = 0; j < k_h; ++j) {
            const int h = kept_heads[(size_t)b * k_h + j];
            if (h < 0 || h >= Hq) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); continue; }
            s_kind[n] = 0; s_idx[n] = h; ++n;
            groups |= 1u << (h / r);
        }
        for (int g = 0; g < Hk; ++g)
            if ((groups >> g) & 1u) { s_kind[n] = 1; s_idx[n] = g; ++n; s_kind[n] = 2; s_idx[n] = g; ++n; }
        s_n = n;
    }
    const T* x = X + ((size_t)b * Tlen + t) * D;
    for (int e = threadIdx.x; e < D; e += blockDim.x) s_x[e] = to_f32<T>(x[e]);
    __syncthreads();
    const int total = s_n * d;
    for (int o = threadIdx.x; o < total; o += blockDim.x) {
        const int sl = o / d, c = o % d;
        const int kind = s_kind[sl], idx = s_idx[sl];
        const T* W = kind == 0 ? WQ : (kind == 1 ? WK : WV);
        const int ld = (kind == 0 ? Hq : Hk) * d;
        const int col = idx * d + c;
        float acc = 0.f;
        for (int e = 0; e < D; ++e) acc = fmaf(s_x[e], to_f32<T>(W[(size_t)e * ld + col]), acc);
        T* dst = kind == 0 ? Q + (((size_t)b * Hq + idx) * Tlen + t) * d
                           : (kind == 1 ? K : V) + (((size_t)b * Hk + idx) * Tlen + t) * d;
        dst[c] = from_f32<T>(acc);
    }
}

template <typename T>
__global__ void __launch_bounds__(kProjThreads)
project_out_kernel(const T* __restrict__ A, const T* __restrict__ WO, const int32_t* __restrict__ kept_heads,
                   const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks, int Tlen, int D, int Hq,
                   int d, int k_h, T* __restrict__ out, unsigned int* status) {
    extern __shared__ float s_a[];                 // [k_h * d]
    __shared__ int s_h[64];
    const int b = blockIdx.x / Tlen, t = blockIdx.x % Tlen;
    T* o = out + ((size_t)b * Tlen + t) * D;
    const int m = ids[t];
    if (m < 0 || m >= 32 || !((masks[b] >> m) & 1u)) {             // absent token: zero row
        for (int e = threadIdx.x; e < D; e += blockDim.x) o[e] = from_f32<T>(0.f);
        return;
    }
    for (int j = threadIdx.x; j < k_h; j += blockDim.x) {
        int h = kept_heads[(size_t)b * k_h + j];
        if (h < 0 || h >= Hq) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); h = -1; }
        s_h[j] = h;
    }
    for (int i = threadIdx.x; i < k_h * d; i += blockDim.x)
        s_a[i] = to_f32<T>(A[(((size_t)b * k_h + i / d) * Tlen + t) * d + i % d]);
    __syncthreads();
    for (int e = threadIdx.x; e < D; e += blockDim.x) {
        float acc = 0.f;
        for (int j = 0; j < k_h; ++j) {
            const int h = s_h[j];
            if (h < 0) continue;
            for (int c = 0; c < d; ++c) acc = fmaf(s_a[j * d + c], to_f32<T>(WO[(size_t)(h * d + c) * D + e]), acc);
        }
        o[e] = from_f32<T>(acc);
    }
}

}  // namespace

int launch_project_qkv_generic(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st) {
    const sentry_proj_desc& d = a.d;
    const unsigned grid = (unsigned)((size_t)d.B * d.T);
    const size_t smem = (size_t)d.D * sizeof(float);
    LaunchScope ls(ctx, KS_PROJ_QKV, st);
    if (d.dtype == SENTRY_F32)
        project_qkv_kernel<float><<<grid, kProjThreads, smem, st>>>(
            (const float*)a.X, (const float*)a.WQ, (const float*)a.WK, (const float*)a.WV, a.kept_heads, a.ids, a.masks,
            d.T, d.D, d.Hq, d.Hk, d.d, d.k_h, (float*)a.Q, (float*)a.K, (float*)a.V, a.status);
    else if (d.dtype == SENTRY_F16)
        project_qkv_kernel<__half><<<grid, kProjThreads, smem, st>>>(
            (const __half*)a.X, (const __half*)a.WQ, (const __half*)a.WK, (const __half*)a.WV, a.kept_heads, a.ids,
            a.masks, d.T, d.D, d.Hq, d.Hk, d.d, d.k_h, (__half*)a.Q, (__half*)a.K, (__half*)a.V, a.status);
    else
        project_qkv_kernel<__nv_bfloat16><<<grid, kProjThreads, smem, st>>>(
            (const __nv_bfloat16*)a.X, (const __nv_bfloat16*)a.WQ, (const __nv_bfloat16*)a.WK,
            (const __nv_bfloat16*)a.WV, a.kept_heads, a.ids, a.masks, d.T, d.D, d.Hq, d.Hk, d.d, d.k_h,
            (__nv_bfloat16*)a.Q, (__nv_bfloat16*)a.K, (__nv_bfloat16*)a.V, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

int launch_project_out_generic(sentry_ctx* ctx, const ProjArgs& a, cudaStream_t st) {
    const sentry_proj_desc& d = a.d;
    const unsigned grid = (unsigned)((size_t)d.B * d.T);
    const size_t smem = (size_t)d.k_h * d.d * sizeof(float);
    LaunchScope ls(ctx, KS_PROJ_OUT, st);
    if (d.dtype == SENTRY_F32)
        project_out_kernel<float><<<grid, kProjThreads, smem, st>>>(
            (const float*)a.A, (const float*)a.WO, a.kept_heads, a.ids, a.masks, d.T, d.D, d.Hq, d.d, d.k_h,
            (float*)a.out, a.status);
    else if (d.dtype == SENTRY_F16)
        project_out_kernel<__half><<<grid, kProjThreads, smem, st>>>(
            (const __half*)a.A, (const __half*)a.WO, a.kept_heads, a.ids, a.masks, d.T, d.D, d.Hq, d.d, d.k_h,
            (__half*)a.out, a.status);
    else
        project_out_kernel<__nv_bfloat16><<<grid, kProjThreads, smem, st>>>(
            (const __nv_bfloat16*)a.A, (const __nv_bfloat16*)a.WO, a.kept_heads, a.ids, a.masks, d.T, d.D, d.Hq, d.d,
            d.k_h, (__nv_bfloat16*)a.out, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

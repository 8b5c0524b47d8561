// SentryAttend (Section 4.4, Eq. 6), reference-precision kernels on the plain
// fp32 ALUs.  They serve the fp32 workload (tensor cores would not meet its
// tolerance) and any bf16 shape the tensor-core path does not take.
//
//   score   M_i = max_{j in S_i} s_ij - mean_{j in S_i} s_ij  for every present query
//   select  the U queries with the largest M_i (ties -> lower index)
//   core    Eq. 6 on the active rows, mean(V_g) on the other present rows,
//           zeros on rows of absent-modality tokens
#include <math.h>

#include "common.cuh"

namespace {

constexpr int kScoreThreads = 128;
constexpr int kCoreThreads = 128;

template <typename T, int D>
__device__ __forceinline__ void load_row(const T* __restrict__ p, float (&r)[D]) {
    if constexpr (sizeof(T) == 4) {
        const float4* v = reinterpret_cast<const float4*>(p);
#pragma unroll
        for (int i = 0; i < D / 4; ++i) {
            float4 x = v[i];
            r[4 * i] = x.x; r[4 * i + 1] = x.y; r[4 * i + 2] = x.z; r[4 * i + 3] = x.w;
        }
    } else {
        const uint4* v = reinterpret_cast<const uint4*>(p);
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            uint4 x = v[i];
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if constexpr (__is_same(T, __half)) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
                    r[8 * i + 2 * j] = f.x;
                    r[8 * i + 2 * j + 1] = f.y;
                } else {   // bf16: the upper half of an fp32
                    r[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
                    r[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                }
            }
        }
    }
}

// grid (ceil(T/threads), B*k_h).  mscore[(b*k_h+kh)*T + p] for p < T_v.
template <typename T, int D>
__global__ void __launch_bounds__(kScoreThreads)
attend_score_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                    const int32_t* __restrict__ kept_heads, const int32_t* __restrict__ ids,
                    const uint32_t* __restrict__ masks, const int32_t* __restrict__ table,
                    const int64_t* __restrict__ offsets, int n_subsets, int Tlen, int Hq, int Hk,
                    int k_h, int c, int score_mode, float* __restrict__ mscore,
                    unsigned int* status) {
    extern __shared__ uint16_t s_valid[];
    __shared__ int red[66];
    const int bh = blockIdx.x, b = bh / k_h;
    const uint32_t mask = masks[b];
    const int Tv = block_build_valid(ids, Tlen, mask, s_valid, red);
    if (Tv == 0) return;
    const int p = blockIdx.y * blockDim.x + threadIdx.x;
    if (blockIdx.y * blockDim.x >= Tv) return;
    const int h = kept_heads[bh];
    if (h < 0 || h >= Hq) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
        return;
    }
    const int g = h / (Hq / Hk);
    const int n_s = sentry_num_active(Tv, c);
    const int32_t* tbl = nullptr;
    if (score_mode != 1) {
        if (mask >= (uint32_t)n_subsets || offsets[mask] < 0) {
            if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            return;
        }
        tbl = table + offsets[mask];
    }
    if (p >= Tv) return;
    const T* Qh = Q + ((size_t)b * Hq + h) * Tlen * D;
    const T* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    float q[D], kr[D];
    load_row<T, D>(Qh + (size_t)s_valid[p] * D, q);
    const float scale = 1.0f / sqrtf((float)D);
    const int cnt = (score_mode != 1) ? n_s : Tv;
    float mx = -INFINITY, sum = 0.f;
    for (int a = 0; a < cnt; ++a) {
        int pj = (score_mode == 0) ? tbl[(size_t)p * n_s + a] : (score_mode == 2 ? tbl[(size_t)a * Tv + p] : a);
        if (pj < 0 || pj >= Tv) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); pj = 0; }
        load_row<T, D>(Kg + (size_t)s_valid[pj] * D, kr);
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < D; ++e) dot = fmaf(q[e], kr[e], dot);
        dot *= scale;
        mx = fmaxf(mx, dot);
        sum += dot;
    }
    mscore[(size_t)bh * Tlen + p] = mx - sum / (float)cnt;
}

// grid B*k_h.  active[bh, 0..U) = token indices of the U best positions, ascending; rest -1.
__global__ void __launch_bounds__(256)
attend_select_kernel(const float* __restrict__ mscore, const int32_t* __restrict__ ids,
                     const uint32_t* __restrict__ masks, int Tlen, int k_h, int c, int U_max,
                     int32_t* __restrict__ active, unsigned int* status) {
    extern __shared__ uint8_t s_raw[];
    __shared__ int red[66];
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(s_raw);
    uint32_t* s_keys = reinterpret_cast<uint32_t*>(s_raw + (((size_t)Tlen * 2 + 15) / 16) * 16);
    const int bh = blockIdx.x, b = bh / k_h;
    const int Tv = block_build_valid(ids, Tlen, masks[b], s_valid, red);
    int32_t* out = active + (size_t)bh * U_max;
    const int U = sentry_num_active(Tv, c);
    for (int i = U + threadIdx.x; i < U_max; i += blockDim.x) out[i] = -1;
    if (Tv == 0) {
        if (threadIdx.x == 0) atomicOr(status, SENTRY_STATUS_BIT_EMPTY_MASK);
        return;
    }
    for (int p = threadIdx.x; p < Tv; p += blockDim.x)
        s_keys[p] = sentry_order_key(mscore[(size_t)bh * Tlen + p]);
    __syncthreads();
    block_select_topk(s_keys, Tv, U, out, s_valid, red);
}

// grid B*k_h.  O[bh, t, :] for every t.
template <typename T, int D>
__global__ void __launch_bounds__(kCoreThreads)
attend_core_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                   const int32_t* __restrict__ kept_heads, const int32_t* __restrict__ ids,
                   const uint32_t* __restrict__ masks, const int32_t* __restrict__ active,
                   int Tlen, int Hq, int Hk, int k_h, int c, int U_max, T* __restrict__ O,
                   unsigned int* status) {
    extern __shared__ uint8_t s_raw[];
    __shared__ int red[66];
    __shared__ float s_ctx[D];
    uint16_t* s_valid = reinterpret_cast<uint16_t*>(s_raw);
    // per token: 0 = absent modality, 1 = present & filled with the context vector, 2 = active
    uint8_t* s_kind = s_raw + (((size_t)Tlen * 2 + 15) / 16) * 16;
    const int bh = blockIdx.x, b = bh / k_h;
    const int Tv = block_build_valid(ids, Tlen, masks[b], s_valid, red);
    T* Oh = O + (size_t)bh * Tlen * D;
    const int h = kept_heads[bh];
    if (Tv == 0 || h < 0 || h >= Hq) {
        for (size_t i = threadIdx.x; i < (size_t)Tlen * D; i += blockDim.x) Oh[i] = from_f32<T>(0.f);
        if (threadIdx.x == 0)
            atomicOr(status, Tv == 0 ? SENTRY_STATUS_BIT_EMPTY_MASK : SENTRY_STATUS_BIT_BAD_INDEX);
        return;
    }
    const int g = h / (Hq / Hk);
    const T* Qh = Q + ((size_t)b * Hq + h) * Tlen * D;
    const T* Kg = K + ((size_t)b * Hk + g) * Tlen * D;
    const T* Vg = V + ((size_t)b * Hk + g) * Tlen * D;
    for (int t = threadIdx.x; t < Tlen; t += blockDim.x) s_kind[t] = 0;
    __syncthreads();
    for (int p = threadIdx.x; p < Tv; p += blockDim.x) s_kind[s_valid[p]] = 1;
    __syncthreads();
    const int32_t* act = active + (size_t)bh * U_max;
    for (int a = threadIdx.x; a < U_max; a += blockDim.x) {
        const int t = act[a];
        if (t < 0) continue;
        if (t >= Tlen || s_kind[t] == 0) { atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX); continue; }
        s_kind[t] = 2;
    }
    // context vector: mean of V_g over present keys
    if (threadIdx.x < D) {
        float acc = 0.f;
        for (int pj = 0; pj < Tv; ++pj) acc += to_f32<T>(Vg[(size_t)s_valid[pj] * D + threadIdx.x]);
        s_ctx[threadIdx.x] = acc / (float)Tv;
    }
    __syncthreads();

    // active rows: one warp per row, lanes stride the present keys (online softmax per lane,
    // merged across the warp at the end)
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const float scale = 1.0f / sqrtf((float)D);
    for (int a = wid; a < U_max; a += nw) {
        const int t = act[a];
        if (t < 0 || t >= Tlen || s_kind[t] != 2) continue;
        float q[D], kr[D], acc[D];
        load_row<T, D>(Qh + (size_t)t * D, q);
#pragma unroll
        for (int e = 0; e < D; ++e) acc[e] = 0.f;
        float m = -INFINITY, l = 0.f;
        for (int pj = lane; pj < Tv; pj += 32) {
            const size_t roff = (size_t)s_valid[pj] * D;
            load_row<T, D>(Kg + roff, kr);
            float dot = 0.f;
#pragma unroll
            for (int e = 0; e < D; ++e) dot = fmaf(q[e], kr[e], dot);
            dot *= scale;
            const float m_new = fmaxf(m, dot);
            const float corr = expf(m - m_new);   // exp(-inf) = 0 on the first key
            const float pexp = expf(dot - m_new);
            load_row<T, D>(Vg + roff, kr);
            l = l * corr + pexp;
#pragma unroll
            for (int e = 0; e < D; ++e) acc[e] = fmaf(pexp, kr[e], acc[e] * corr);
            m = m_new;
        }
        float m_all = m;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, o));
        const float w = (m == -INFINITY) ? 0.f : expf(m - m_all);
        l *= w;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        const float inv = 1.0f / l;
#pragma unroll
        for (int e = 0; e < D; ++e) {
            float v = acc[e] * w;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            acc[e] = v * inv;
        }
        // lane e writes element e (D <= 64 -> two rounds)
#pragma unroll
        for (int e = 0; e < D; ++e)
            if ((e & 31) == lane) Oh[(size_t)t * D + e] = from_f32<T>(acc[e]);
    }
    // fill rows and zero rows
    for (size_t i = threadIdx.x; i < (size_t)Tlen * D; i += blockDim.x) {
        const int t = (int)(i / D), e = (int)(i % D);
        const uint8_t kind = s_kind[t];
        if (kind == 2) continue;
        Oh[i] = from_f32<T>(kind == 1 ? s_ctx[e] : 0.f);
    }
}

template <typename T, int D>
int launch_typed(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    const sentry_attend_desc& d = a.d;
    const int BH = d.B * d.k_h;
    const size_t valid_bytes = (((size_t)d.T * 2 + 15) / 16) * 16;
    if (!a.selection_given) {
        {
            auto kern = attend_score_kernel<T, D>;
            if (valid_bytes > 48 * 1024)
                SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)valid_bytes));
            dim3 grid(BH, (d.T + kScoreThreads - 1) / kScoreThreads);   // (sample, head) on x: no 65535 limit
            LaunchScope ls(ctx, KS_ATT_SCORE, st);
            kern<<<grid, kScoreThreads, valid_bytes, st>>>(
                (const T*)a.Q, (const T*)a.K, a.kept_heads, a.ids, a.masks, a.sample_table,
                a.sample_offsets, a.n_subsets, d.T, d.Hq, d.Hk, d.k_h, d.c, d.score_mode, a.mscore,
                a.status);
        }
        SENTRY_CUDA_TRY(cudaGetLastError());
        {
            const size_t smem = valid_bytes + (size_t)d.T * 4;
            if (smem > 48 * 1024)
                SENTRY_CUDA_TRY(cudaFuncSetAttribute(attend_select_kernel,
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)smem));
            LaunchScope ls(ctx, KS_ATT_SELECT, st);
            attend_select_kernel<<<BH, 256, smem, st>>>(a.mscore, a.ids, a.masks, d.T, d.k_h, d.c,
                                                         a.U_max, a.active, a.status);
        }
        SENTRY_CUDA_TRY(cudaGetLastError());
    }
    {
        auto kern = attend_core_kernel<T, D>;
        const size_t smem = valid_bytes + (size_t)d.T;
        if (smem > 48 * 1024)
            SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem));
        LaunchScope ls(ctx, KS_ATT_CORE, st);
        kern<<<BH, kCoreThreads, smem, st>>>((const T*)a.Q, (const T*)a.K, (const T*)a.V,
                                              a.kept_heads, a.ids, a.masks, a.active, d.T, d.Hq,
                                              d.Hk, d.k_h, d.c, a.U_max, (T*)a.O, a.status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

}  // namespace

int launch_attend_generic(sentry_ctx* ctx, const AttendArgs& a, cudaStream_t st) {
    const bool f32 = a.d.dtype == SENTRY_F32, f16 = a.d.dtype == SENTRY_F16;
    switch (a.d.d) {
        case 16: return f32 ? launch_typed<float, 16>(ctx, a, st) : f16 ? launch_typed<__half, 16>(ctx, a, st) : launch_typed<__nv_bfloat16, 16>(ctx, a, st);
        case 32: return f32 ? launch_typed<float, 32>(ctx, a, st) : f16 ? launch_typed<__half, 32>(ctx, a, st) : launch_typed<__nv_bfloat16, 32>(ctx, a, st);
        case 64: return f32 ? launch_typed<float, 64>(ctx, a, st) : f16 ? launch_typed<__half, 64>(ctx, a, st) : launch_typed<__nv_bfloat16, 64>(ctx, a, st);
        default: return SENTRY_ERR_UNSUPPORTED;
    }
}

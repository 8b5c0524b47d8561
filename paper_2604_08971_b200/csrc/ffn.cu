// Channel-compacted FFN (Section 4.6): y = gelu(x W1[:, N]) W2[N, :].
// This file holds the row plan, the weight gather ("materialising" W1', W2')
// and the plain-ALU fp32-accumulate kernel; the tensor-core kernel for bf16
// lives in ffn_tc.cu and shares the plan.
#include <math.h>

#include "common.cuh"
#include <cuda_fp8.h>

#include "ffn_plan.cuh"

int launch_ffn_tc(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1c, void* w2c,
                  int kc_pad, int max_tiles, cudaStream_t st);  // ffn_tc.cu
bool ffn_tc_supported(const sentry_ffn_desc& d);
int ffn_tc_kc_pad(int D, int k_c);

namespace {

constexpr int kGenericTileRows = 16;
constexpr int kGenericThreads = 256;
constexpr int kTcTileRows = 128;

// One launch prepares everything the main kernel needs.  Block ranges:
//   [0, B)              row table of sample b: every block finds by itself where its sample's
//                       rows start (a scan over all samples' lists and present-row counts, so no
//                       separate planning launch is needed); block 0 also writes the per-list
//                       offsets and tile counts
//   [B, B + B*zsplit)   zero rows of Y for the absent tokens of a sample (slices of its rows)
//   [.., + prepack)     the weight gather, which "materialises" the pruned W1', W2' per list:
//     layout 0 (plain-ALU kernel): W1g [l][D][kc_pad], W2g [l][kc_pad][D]
//     layout 1 (tensor-core kernel, both K-major): W1c [l][kc_pad][D], W2c [l][D][kc_pad]
//     columns / rows n >= k_c are zero.
template <typename T>
__global__ void __launch_bounds__(256)
ffn_prepare_kernel(const int32_t* __restrict__ ids, const uint32_t* __restrict__ masks,
                   const int32_t* __restrict__ list_of_sample, int B, int Tlen, int zsplit,
                   int tile_rows, FfnPlan p, uint8_t* __restrict__ Y,
                   const T* __restrict__ W1, const T* __restrict__ W2,
                   const int32_t* __restrict__ kept, int n_lists, int D, int F, int k_c, int kc_pad,
                   int layout, size_t w_stride, T* __restrict__ out1, T* __restrict__ out2,
                   unsigned int* status) {
    // w_stride: elements between the weight matrices of consecutive lists (0: every list gathers
    // from the same W1, W2; D*F: list l has its own, as the experts of a Sparse-MoE block do)
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    if ((int)blockIdx.x < B) {
        __shared__ int s_cnt[32];
        __shared__ int red[66];
        const int b = blockIdx.x;
        if (threadIdx.x < 32) s_cnt[threadIdx.x] = 0;
        __syncthreads();
        if (ids != nullptr) {
            for (int t = threadIdx.x; t < Tlen; t += blockDim.x) {
                const int m = ids[t];
                if (m >= 0 && m < 32) atomicAdd(&s_cnt[m], 1);
                else if (b == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
            }
            __syncthreads();
        }
        auto present_rows = [&](int bb) {
            if (ids == nullptr) return Tlen;
            uint32_t mask = masks[bb];
            int n = 0;
            while (mask) { const int m = __ffs(mask) - 1; n += s_cnt[m]; mask &= mask - 1; }
            return n;
        };
        auto list_of = [&](int bb) {
            int l = list_of_sample ? list_of_sample[bb] : 0;
            if (l < 0 || l >= n_lists) {
                if (b == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
                l = 0;
            }
            return l;
        };
        // rows of all samples in earlier lists, and of earlier samples in this sample's list
        const int my_list = list_of(b);
        int before = 0;
        for (int bb = threadIdx.x; bb < B; bb += blockDim.x) {
            const int l = list_of(bb);
            if (l < my_list || (l == my_list && bb < b)) before += present_rows(bb);
        }
        before = block_sum_int(before, red);
        if (threadIdx.x == 0) p.sample_row0[b] = before;
        if (b == 0) {
            // per-list totals -> list offsets and tile counts (lists are few: one pass each)
            int row0 = 0, tile0 = 0;
            for (int l = 0; l < n_lists; ++l) {
                int rows = 0;
                for (int bb = threadIdx.x; bb < B; bb += blockDim.x)
                    if (list_of(bb) == l) {
                        const int r = present_rows(bb);
                        rows += r;
                        if (r == 0) atomicOr(status, SENTRY_STATUS_BIT_EMPTY_MASK);
                    }
                rows = block_sum_int(rows, red);
                if (threadIdx.x == 0) { p.list_row0[l] = row0; p.tile_start[l] = tile0; }
                row0 += rows;
                tile0 += (rows + tile_rows - 1) / tile_rows;
            }
            if (threadIdx.x == 0) { p.list_row0[n_lists] = row0; p.tile_start[n_lists] = tile0; }
        }
        // present tokens of this sample, ascending -> row table
        const uint32_t mask = (ids != nullptr) ? masks[b] : 0xffffffffu;
        int32_t* rows = p.rowidx + before;
        int base = 0;
        for (int t0 = 0; t0 < Tlen; t0 += blockDim.x) {
            const int t = t0 + threadIdx.x;
            bool ok = false;
            if (t < Tlen) {
                if (ids == nullptr) ok = true;
                else { const int m = ids[t]; ok = (m >= 0 && m < 32) && ((mask >> m) & 1u); }
            }
            const unsigned bm = __ballot_sync(0xffffffffu, ok);
            __syncthreads();
            if (lane == 0) red[wid] = __popc(bm);
            __syncthreads();
            int pos = base, tot = 0;
            for (int w = 0; w < nw; ++w) { if (w < wid) pos += red[w]; tot += red[w]; }
            if (ok) rows[pos + __popc(bm & ((1u << lane) - 1u))] = b * Tlen + t;
            base += tot;
        }
        return;
    }
    size_t pb = (size_t)blockIdx.x - B;
    const size_t zero_blocks = (ids != nullptr) ? (size_t)B * zsplit : 0;
    if (pb < zero_blocks) {
        // zero the rows of absent tokens, 16 bytes per store
        const int b = (int)(pb / zsplit), part = (int)(pb % zsplit);
        const uint32_t mask = masks[b];
        const int vpr = D * (int)sizeof(T) / 16;
        const int total = Tlen * vpr;
        const int per = (total + zsplit - 1) / zsplit;
        const int end = min(total, (part + 1) * per);
        uint4* Yb = reinterpret_cast<uint4*>(Y + (size_t)b * Tlen * D * sizeof(T));
        for (int i = part * per + threadIdx.x; i < end; i += blockDim.x) {
            const int m = ids[i / vpr];
            const bool present = (m >= 0 && m < 32) && ((mask >> m) & 1u);
            if (!present) Yb[i] = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    pb -= zero_blocks;
    if (layout == 1) {
        // K-major copies for the tensor-core kernel, one 32-channel x 64-column tile per block,
        // transposed through shared memory so that both the gather and the store touch whole
        // sectors:  W1c[l][n][e] = W1[e][N[n]],  W2c[l][e][n] = W2[N[n]][e].
        __shared__ T s_tile[64][33];
        __shared__ int s_ch[32];
        const int tiles_n = kc_pad / 32, tiles_e = D / 64;
        const size_t per_list = (size_t)tiles_n * tiles_e;
        const int which = (int)(pb / (per_list * n_lists));
        pb -= (size_t)which * per_list * n_lists;
        const int l = (int)(pb / per_list);
        const int tn = (int)((pb % per_list) / tiles_e), te = (int)(pb % tiles_e);
        const int n0 = tn * 32, e0 = te * 64;
        const T* W1l = W1 + (size_t)l * w_stride;
        const T* W2l = W2 + (size_t)l * w_stride;
        const int tx = threadIdx.x & 31, wy = threadIdx.x >> 5;   // 8 warps
        if (threadIdx.x < 32) {
            const int n = n0 + threadIdx.x;
            int ch = -1;
            if (n < k_c) {
                ch = kept[(size_t)l * k_c + n];
                if (ch < 0 || ch >= F) {
                    if (which == 0 && te == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
                    ch = -1;
                }
            }
            s_ch[threadIdx.x] = ch;
        }
        __syncthreads();
        const T zero = from_f32<T>(0.f);
        if (which == 0) {
            const int ch = s_ch[tx];
            for (int ee = wy; ee < 64; ee += 8)
                s_tile[ee][tx] = ch >= 0 ? W1l[(size_t)(e0 + ee) * F + ch] : zero;
            __syncthreads();
            T* dst = out1 + ((size_t)l * kc_pad + n0) * D + e0;
            for (int nn = wy; nn < 32; nn += 8) {
                dst[(size_t)nn * D + tx] = s_tile[tx][nn];
                dst[(size_t)nn * D + 32 + tx] = s_tile[32 + tx][nn];
            }
        } else {
            for (int nn = wy; nn < 32; nn += 8) {
                const int ch = s_ch[nn];
                s_tile[tx][nn] = ch >= 0 ? W2l[(size_t)ch * D + e0 + tx] : zero;
                s_tile[32 + tx][nn] = ch >= 0 ? W2l[(size_t)ch * D + e0 + 32 + tx] : zero;
            }
            __syncthreads();
            T* dst = out2 + ((size_t)l * D + e0) * kc_pad + n0;
            for (int ee = wy; ee < 64; ee += 8) dst[(size_t)ee * kc_pad + tx] = s_tile[ee][tx];
        }
        return;
    }
    const size_t per = (size_t)kc_pad * D;
    const size_t blocks_per = (per + 255) / 256;
    const int which = (int)(pb / (blocks_per * n_lists));
    pb -= (size_t)which * blocks_per * n_lists;
    const int l = (int)(pb / blocks_per);
    const size_t i = (pb % blocks_per) * 256 + threadIdx.x;
    if (i >= per) return;
    const int32_t* N = kept + (size_t)l * k_c;
    if (which == 0) {
        // W1: destination-major index so that writes coalesce
        int n, e;
        if (layout == 0) { e = (int)(i / kc_pad); n = (int)(i % kc_pad); }
        else             { n = (int)(i / D);      e = (int)(i % D); }
        T v = from_f32<T>(0.f);
        if (n < k_c) {
            const int ch = N[n];
            if (ch >= 0 && ch < F) v = W1[(size_t)l * w_stride + (size_t)e * F + ch];
            else if (e == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
        }
        out1[(size_t)l * per + i] = v;
    } else {
        int n, e;
        if (layout == 0) { n = (int)(i / D);      e = (int)(i % D); }
        else             { e = (int)(i / kc_pad); n = (int)(i % kc_pad); }
        T v = from_f32<T>(0.f);
        if (n < k_c) {
            const int ch = N[n];
            if (ch >= 0 && ch < F) v = W2[(size_t)l * w_stride + (size_t)ch * D + e];
        }
        out2[(size_t)l * per + i] = v;
    }
}

// The weight gather from FP8 storage: W1q [D,F] and W2q [F,D] hold e4m3 codes (4 exponent bits, 3
// fraction bits, bias 7, no infinities), each with one fp32 scale; element = decode(code) * scale,
// rounded once to the compute type T.  Same destination layouts as the gather above; a one-off
// (materialise-once) step, so one thread per destination element is enough.
template <typename T>
__global__ void __launch_bounds__(256)
ffn_prepack_fp8_kernel(const uint8_t* __restrict__ W1q, const uint8_t* __restrict__ W2q, float s1, float s2,
                       const int32_t* __restrict__ kept, int n_lists, int D, int F, int k_c, int kc_pad,
                       int layout, T* __restrict__ out1, T* __restrict__ out2, unsigned int* status) {
    const size_t per = (size_t)kc_pad * D;
    const size_t blocks_per = (per + 255) / 256;
    size_t pb = blockIdx.x;
    const int which = (int)(pb / (blocks_per * n_lists));
    pb -= (size_t)which * blocks_per * n_lists;
    const int l = (int)(pb / blocks_per);
    const size_t i = (pb % blocks_per) * 256 + threadIdx.x;
    if (i >= per) return;
    const int32_t* N = kept + (size_t)l * k_c;
    auto decode = [](uint8_t code) {
        __nv_fp8_e4m3 q;
        q.__x = code;
        return float(q);
    };
    int n, e;
    if (which == 0) {
        if (layout == 0) { e = (int)(i / kc_pad); n = (int)(i % kc_pad); }
        else             { n = (int)(i / D);      e = (int)(i % D); }
    } else {
        if (layout == 0) { n = (int)(i / D);      e = (int)(i % D); }
        else             { e = (int)(i / kc_pad); n = (int)(i % kc_pad); }
    }
    T v = from_f32<T>(0.f);
    if (n < k_c) {
        const int ch = N[n];
        if (ch >= 0 && ch < F)
            v = which == 0 ? from_f32<T>(decode(W1q[(size_t)e * F + ch]) * s1) : from_f32<T>(decode(W2q[(size_t)ch * D + e]) * s2);
        else if (which == 0 && e == 0) atomicOr(status, SENTRY_STATUS_BIT_BAD_INDEX);
    }
    (which == 0 ? out1 : out2)[(size_t)l * per + i] = v;
}

__device__ __forceinline__ float gelu_erf(float z) {
    return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f));
}

// Plain-ALU fused pair on a tile of 16 present rows.  grid = tile upper bound.
template <typename T>
__global__ void __launch_bounds__(kGenericThreads)
ffn_generic_kernel(const T* __restrict__ X, const T* __restrict__ W1g, const T* __restrict__ W2g,
                   FfnPlan plan, int n_lists, int Tlen, int D, int k_c, int kc_pad,
                   T* __restrict__ Y) {
    extern __shared__ float s_f[];
    float* s_x = s_f;                                  // [16][D]
    float* s_h = s_f + (size_t)kGenericTileRows * D;   // [16][256]
    __shared__ long long s_row[kGenericTileRows], s_out[kGenericTileRows];
    int l, row0, n_rows;
    if (!ffn_tile_lookup(plan, n_lists, blockIdx.x, kGenericTileRows, l, row0, n_rows)) return;
    if (threadIdx.x < kGenericTileRows)
        s_row[threadIdx.x] = threadIdx.x < n_rows ? (long long)plan.rowidx[row0 + threadIdx.x] : -1;
    if (threadIdx.x < kGenericTileRows)
        s_out[threadIdx.x] = threadIdx.x < n_rows
                                 ? (long long)(plan.rowout ? plan.rowout : plan.rowidx)[row0 + threadIdx.x] : -1;
    __syncthreads();
    for (int i = threadIdx.x; i < kGenericTileRows * D; i += blockDim.x) {
        const int r = i / D, e = i % D;
        s_x[i] = s_row[r] >= 0 ? to_f32<T>(X[(size_t)s_row[r] * D + e]) : 0.f;
    }
    const T* w1 = W1g + (size_t)l * D * kc_pad;
    const T* w2 = W2g + (size_t)l * kc_pad * D;
    constexpr int kMaxSlots = 4;  // D <= 1024
    float y[kMaxSlots][kGenericTileRows];
#pragma unroll
    for (int s = 0; s < kMaxSlots; ++s)
#pragma unroll
        for (int r = 0; r < kGenericTileRows; ++r) y[s][r] = 0.f;
    __syncthreads();
    for (int c0 = 0; c0 < k_c; c0 += kGenericThreads) {
        const int n = c0 + threadIdx.x;
        float hacc[kGenericTileRows];
#pragma unroll
        for (int r = 0; r < kGenericTileRows; ++r) hacc[r] = 0.f;
        if (n < k_c) {
            for (int e = 0; e < D; ++e) {
                const float w = to_f32<T>(w1[(size_t)e * kc_pad + n]);
#pragma unroll
                for (int r = 0; r < kGenericTileRows; ++r) hacc[r] = fmaf(s_x[r * D + e], w, hacc[r]);
            }
        }
#pragma unroll
        for (int r = 0; r < kGenericTileRows; ++r)
            s_h[r * kGenericThreads + threadIdx.x] = (n < k_c) ? gelu_erf(hacc[r]) : 0.f;
        __syncthreads();
        const int cn = min(kGenericThreads, k_c - c0);
#pragma unroll
        for (int s = 0; s < kMaxSlots; ++s) {
            const int e = s * kGenericThreads + threadIdx.x;
            if (e < D) {
                for (int j = 0; j < cn; ++j) {
                    const float w = to_f32<T>(w2[(size_t)(c0 + j) * D + e]);
#pragma unroll
                    for (int r = 0; r < kGenericTileRows; ++r)
                        y[s][r] = fmaf(s_h[r * kGenericThreads + j], w, y[s][r]);
                }
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int s = 0; s < kMaxSlots; ++s) {
        const int e = s * kGenericThreads + threadIdx.x;
        if (e < D) {
#pragma unroll
            for (int r = 0; r < kGenericTileRows; ++r)
                if (s_out[r] >= 0) Y[(size_t)s_out[r] * D + e] = from_f32<T>(y[s][r]);
        }
    }
}

struct FfnWs {
    FfnPlan plan;
    void *w1p, *w2p;
    bool ok;
    size_t used;
};

// One of W1', W2' (all lists), rounded so that the second starts 256-byte aligned.
size_t packed_half_bytes(const sentry_ffn_desc& d, int kc_pad) {
    const size_t esz = d.dtype == SENTRY_F32 ? 4 : (d.dtype == SENTRY_FP8_E4M3 ? 1 : 2);
    return align_up((size_t)d.n_lists * kc_pad * d.D * esz, 256);
}

// Row plan (and, unless the caller brings materialised weights, W1' and W2') from the workspace.
FfnWs carve(const sentry_ffn_desc& d, int kc_pad, void* ws, size_t bytes, bool with_weights) {
    WsAlloc a(ws, bytes);
    FfnWs w;
    w.plan.sample_row0 = a.take<int32_t>(d.B);
    w.plan.list_row0 = a.take<int32_t>(d.n_lists + 1);
    w.plan.tile_start = a.take<int32_t>(d.n_lists + 1);
    w.plan.rowidx = a.take<int32_t>((size_t)d.B * d.T);
    w.plan.rowout = nullptr;
    w.w1p = w.w2p = nullptr;
    if (with_weights) {
        w.w1p = a.take<uint8_t>(packed_half_bytes(d, kc_pad));
        w.w2p = a.take<uint8_t>(packed_half_bytes(d, kc_pad));
    }
    w.ok = a.ok;
    w.used = a.off;
    return w;
}

int kc_pad_for(const sentry_ffn_desc& d) {
    if (ffn_tc_supported(d)) return ffn_tc_kc_pad(d.D, d.k_c);
    return (d.k_c + 7) / 8 * 8;
}

}  // namespace

size_t ffn_workspace_bytes(const sentry_ffn_desc& d) {
    return carve(d, kc_pad_for(d), nullptr, 0, true).used + 256;
}

size_t ffn_packed_bytes(const sentry_ffn_desc& d) { return 2 * packed_half_bytes(d, kc_pad_for(d)); }

// The weight gather alone: W1' = W1[:, N], W2' = W2[N, :] for every list into `packed`.
// (The gather moves elements and writes zeros, no arithmetic: fp16 data goes through the 16-bit
// instantiation unchanged.)
int launch_ffn_prepack(sentry_ctx* ctx, const FfnArgs& a, void* packed, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    const bool tc = ffn_tc_supported(d);
    const int kc_pad = kc_pad_for(d);
    const size_t per = (size_t)kc_pad * d.D;
    const size_t pack_blocks = tc ? 2 * (size_t)d.n_lists * (kc_pad / 32) * (d.D / 64)
                                  : 2 * (size_t)d.n_lists * ((per + 255) / 256);
    uint8_t* w1p = (uint8_t*)packed;
    uint8_t* w2p = w1p + packed_half_bytes(d, kc_pad);
    FfnPlan none = {};
    none.rowout = nullptr;
    LaunchScope ls(ctx, KS_FFN_PREPARE, st);
    // no row-table and no zero-fill blocks (B = 0, no ids): every block gathers weights
    if (d.dtype == SENTRY_FP8_E4M3) {
        if (!tc) return SENTRY_ERR_UNSUPPORTED;
        ffn_prepare_kernel<uint8_t><<<(unsigned)pack_blocks, 256, 0, st>>>(
            nullptr, nullptr, nullptr, 0, d.T, 1, kTcTileRows, none, nullptr, (const uint8_t*)a.W1, (const uint8_t*)a.W2,
            a.kept, d.n_lists, d.D, d.F, d.k_c, kc_pad, 1, a.w_stride, w1p, w2p, a.status);
    } else if (d.dtype == SENTRY_F32)
        ffn_prepare_kernel<float><<<(unsigned)pack_blocks, 256, 0, st>>>(
            nullptr, nullptr, nullptr, 0, d.T, 1, kGenericTileRows, none, nullptr, (const float*)a.W1,
            (const float*)a.W2, a.kept, d.n_lists, d.D, d.F, d.k_c, kc_pad, 0, a.w_stride, (float*)w1p, (float*)w2p, a.status);
    else
        ffn_prepare_kernel<__nv_bfloat16><<<(unsigned)pack_blocks, 256, 0, st>>>(
            nullptr, nullptr, nullptr, 0, d.T, 1, tc ? kTcTileRows : kGenericTileRows, none, nullptr,
            (const __nv_bfloat16*)a.W1, (const __nv_bfloat16*)a.W2, a.kept, d.n_lists, d.D, d.F, d.k_c, kc_pad,
            tc ? 1 : 0, a.w_stride, (__nv_bfloat16*)w1p, (__nv_bfloat16*)w2p, a.status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

int launch_ffn_prepack_fp8(sentry_ctx* ctx, const sentry_ffn_desc& d, const uint8_t* W1q, const uint8_t* W2q, float s1,
                           float s2, const int32_t* kept, void* packed, cudaStream_t st) {
    const bool tc = ffn_tc_supported(d);
    const int kc_pad = kc_pad_for(d);
    const size_t per = (size_t)kc_pad * d.D;
    const unsigned grid = (unsigned)(2 * (size_t)d.n_lists * ((per + 255) / 256));
    uint8_t* w1p = (uint8_t*)packed;
    uint8_t* w2p = w1p + packed_half_bytes(d, kc_pad);
    const int layout = tc ? 1 : 0;
    LaunchScope ls(ctx, KS_FFN_PREPARE, st);
    if (d.dtype == SENTRY_F32)
        ffn_prepack_fp8_kernel<float><<<grid, 256, 0, st>>>(W1q, W2q, s1, s2, kept, d.n_lists, d.D, d.F, d.k_c, kc_pad,
                                                           layout, (float*)w1p, (float*)w2p, ctx->d_status);
    else if (d.dtype == SENTRY_F16)
        ffn_prepack_fp8_kernel<__half><<<grid, 256, 0, st>>>(W1q, W2q, s1, s2, kept, d.n_lists, d.D, d.F, d.k_c, kc_pad,
                                                            layout, (__half*)w1p, (__half*)w2p, ctx->d_status);
    else
        ffn_prepack_fp8_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(W1q, W2q, s1, s2, kept, d.n_lists, d.D, d.F, d.k_c,
                                                                   kc_pad, layout, (__nv_bfloat16*)w1p,
                                                                   (__nv_bfloat16*)w2p, ctx->d_status);
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

int ffn_kc_pad(const sentry_ffn_desc& d) { return kc_pad_for(d); }
int ffn_tile_rows(const sentry_ffn_desc& d) {
    return ffn_tc_supported(d) ? kTcTileRows : kGenericTileRows;
}

// The fused pair alone, on a row plan and materialised weights that are already in place.
int launch_ffn_main(sentry_ctx* ctx, const FfnArgs& a, const FfnPlan& plan, void* w1p, void* w2p, int kc_pad,
                    int max_tiles, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    const bool tc = ffn_tc_supported(d);
    if (tc) {
        int rc = launch_ffn_tc(ctx, a, plan, w1p, w2p, kc_pad, max_tiles, st);
        if (rc != SENTRY_OK) return rc;
    } else {
        const size_t smem = ((size_t)kGenericTileRows * d.D + kGenericTileRows * kGenericThreads) * 4;
        LaunchScope ls(ctx, KS_FFN_MAIN, st);
        if (d.dtype == SENTRY_F32) {
            auto kern = ffn_generic_kernel<float>;
            if (smem > 48 * 1024)
                SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            kern<<<max_tiles, kGenericThreads, smem, st>>>((const float*)a.X, (const float*)w1p,
                                                            (const float*)w2p, plan, d.n_lists,
                                                            d.T, d.D, d.k_c, kc_pad, (float*)a.Y);
        } else if (d.dtype == SENTRY_F16) {
            auto kern = ffn_generic_kernel<__half>;
            if (smem > 48 * 1024)
                SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            kern<<<max_tiles, kGenericThreads, smem, st>>>(
                (const __half*)a.X, (const __half*)w1p, (const __half*)w2p,
                plan, d.n_lists, d.T, d.D, d.k_c, kc_pad, (__half*)a.Y);
        } else {
            auto kern = ffn_generic_kernel<__nv_bfloat16>;
            if (smem > 48 * 1024)
                SENTRY_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            kern<<<max_tiles, kGenericThreads, smem, st>>>(
                (const __nv_bfloat16*)a.X, (const __nv_bfloat16*)w1p, (const __nv_bfloat16*)w2p,
                plan, d.n_lists, d.T, d.D, d.k_c, kc_pad, (__nv_bfloat16*)a.Y);
        }
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    return SENTRY_OK;
}

// packed == nullptr: gather the weights into the workspace first (every call); otherwise use the
// caller's materialised W1', W2' (launch_ffn_prepack) and only build the row plan.
int launch_ffn(sentry_ctx* ctx, const FfnArgs& a, void* ws, size_t ws_bytes, const void* packed, cudaStream_t st) {
    const sentry_ffn_desc& d = a.d;
    const bool tc = ffn_tc_supported(d);
    const int kc_pad = kc_pad_for(d);
    if (d.dtype == SENTRY_FP8_E4M3 && (packed == nullptr || !tc)) return SENTRY_ERR_UNSUPPORTED;   // FP8: prepacked weights only
    FfnWs w = carve(d, kc_pad, ws, ws_bytes, packed == nullptr);
    if (!w.ok) return SENTRY_ERR_WORKSPACE;
    if (packed != nullptr) {
        w.w1p = const_cast<void*>(packed);
        w.w2p = (uint8_t*)w.w1p + packed_half_bytes(d, kc_pad);
    }
    const int tile_rows = tc ? kTcTileRows : kGenericTileRows;

    {
        const size_t per = (size_t)kc_pad * d.D;
        // enough zero-fill blocks to cover the GPU a few times over when the batch is small
        int zsplit = (4 * ctx->sm_count + d.B - 1) / d.B;
        if (zsplit < 1) zsplit = 1;
        if (zsplit > 32) zsplit = 32;
        const size_t pack_blocks = packed != nullptr ? 0
                                   : (tc ? 2 * (size_t)d.n_lists * (kc_pad / 32) * (d.D / 64)
                                         : 2 * (size_t)d.n_lists * ((per + 255) / 256));
        const size_t grid = (size_t)d.B + (a.ids != nullptr ? (size_t)d.B * zsplit : 0) + pack_blocks;
        LaunchScope ls(ctx, KS_FFN_PREPARE, st);
        if (d.dtype == SENTRY_F32)
            ffn_prepare_kernel<float><<<(unsigned)grid, 256, 0, st>>>(
                a.ids, a.masks, a.list_of_sample, d.B, d.T, zsplit, tile_rows, w.plan, (uint8_t*)a.Y,
                (const float*)a.W1, (const float*)a.W2, a.kept, d.n_lists, d.D, d.F, d.k_c, kc_pad, 0, a.w_stride,
                (float*)w.w1p, (float*)w.w2p, a.status);
        else
            ffn_prepare_kernel<__nv_bfloat16><<<(unsigned)grid, 256, 0, st>>>(
                a.ids, a.masks, a.list_of_sample, d.B, d.T, zsplit, tile_rows, w.plan, (uint8_t*)a.Y,
                (const __nv_bfloat16*)a.W1, (const __nv_bfloat16*)a.W2, a.kept, d.n_lists, d.D, d.F,
                d.k_c, kc_pad, tc ? 1 : 0, a.w_stride, (__nv_bfloat16*)w.w1p, (__nv_bfloat16*)w.w2p, a.status);
    }
    SENTRY_CUDA_TRY(cudaGetLastError());
    const long long rows = (long long)d.B * d.T;
    const int max_tiles = (int)((rows + tile_rows - 1) / tile_rows) + d.n_lists;
    return launch_ffn_main(ctx, a, w.plan, w.w1p, w.w2p, kc_pad, max_tiles, st);
}

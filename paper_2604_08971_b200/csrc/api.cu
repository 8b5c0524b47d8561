// C ABI of libsentry: argument validation, workspace carving and dispatch.
// Everything numerical happens in the kernels of the other translation units.
#include <new>

#include "common.cuh"

namespace {

constexpr size_t kMinWorkspace = 1u << 20;
constexpr int kMaxTokens = 32768;
constexpr int kMaxUnits = 49152;

inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

size_t attend_workspace_bytes(const sentry_attend_desc& d) {
    const int U_max = sentry_num_active(d.T, d.c);
    WsAlloc a(nullptr, 0);
    a.take<float>((size_t)d.B * d.k_h * d.T);
    a.take<int32_t>((size_t)d.B * d.k_h * U_max);
    return a.off + 256;
}

int check_attend_desc(const sentry_attend_desc* d) {
    if (d == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (d->dtype != SENTRY_F32 && d->dtype != SENTRY_BF16 && d->dtype != SENTRY_F16) return SENTRY_ERR_INVALID_ARG;
    if (d->score_mode < 0 || d->score_mode > 2) return SENTRY_ERR_INVALID_ARG;
    if (d->B < 1 || d->T < 1 || d->Hq < 1 || d->Hk < 1 || d->k_h < 1 || d->c < 1)
        return SENTRY_ERR_BAD_SHAPE;
    if (d->Hq % d->Hk != 0 || d->k_h > d->Hq) return SENTRY_ERR_BAD_SHAPE;
    if (d->T > kMaxTokens) return SENTRY_ERR_UNSUPPORTED;
    if (d->d != 16 && d->d != 32 && d->d != 64) return SENTRY_ERR_UNSUPPORTED;
    if ((long long)d->B * d->k_h > 0x7fffffffLL / 4) return SENTRY_ERR_UNSUPPORTED;
    return SENTRY_OK;
}

int check_ffn_desc(const sentry_ffn_desc* d, bool fp8_ok = false) {
    if (d == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (d->dtype == SENTRY_FP8_E4M3) {
        if (!fp8_ok) return SENTRY_ERR_UNSUPPORTED;
    } else if (d->dtype != SENTRY_F32 && d->dtype != SENTRY_BF16 && d->dtype != SENTRY_F16) {
        return SENTRY_ERR_INVALID_ARG;
    }
    if (d->B < 1 || d->T < 1 || d->D < 1 || d->F < 1 || d->k_c < 1 || d->n_lists < 1)
        return SENTRY_ERR_BAD_SHAPE;
    if (d->k_c > d->F) return SENTRY_ERR_BAD_SHAPE;
    if (d->D % 8 != 0 || d->D > 1024 || d->T > 65535 || d->n_lists > 4096)
        return SENTRY_ERR_UNSUPPORTED;
    if ((long long)d->B * d->T > 0x7fffffffLL - 8192) return SENTRY_ERR_UNSUPPORTED;
    return SENTRY_OK;
}

}  // namespace

extern "C" {

int sentry_create(sentry_ctx** out, int device) {
    if (out == nullptr) return SENTRY_ERR_INVALID_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return SENTRY_ERR_CUDA;
    SENTRY_ON_DEVICE(device);
    sentry_ctx* c = new (std::nothrow) sentry_ctx();
    if (c == nullptr) return SENTRY_ERR_CUDA;
    c->device = device;
    c->workspace = nullptr;
    c->workspace_bytes = 0;
    c->last_launches = 0;
    c->profiling = false;
    c->attend_kernel = SENTRY_ATTEND_AUTO;
    c->long_select = SENTRY_LONG_SELECT_AUTO;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return SENTRY_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    if (cudaMalloc((void**)&c->d_status, sizeof(unsigned int)) != cudaSuccess) { delete c; return SENTRY_ERR_CUDA; }
    if (cudaMemset(c->d_status, 0, sizeof(unsigned int)) != cudaSuccess) {
        cudaFree(c->d_status);
        delete c;
        return SENTRY_ERR_CUDA;
    }
    *out = c;
    return SENTRY_OK;
}

int sentry_destroy(sentry_ctx* ctx) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaFree(ctx->d_status);
    for (ProfRec& r : ctx->prof) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    for (cudaEvent_t e : ctx->pool) cudaEventDestroy(e);
    delete ctx;
    return SENTRY_OK;
}

int sentry_profile_enable(sentry_ctx* ctx, int on) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    ctx->profiling = on != 0;
    return SENTRY_OK;
}

int sentry_profile_slots(void) { return KS_COUNT; }

const char* sentry_kernel_name(int slot) {
    static const char* names[KS_COUNT] = {"gate_rows", "gate_expand", "attend_score", "attend_select",
                                          "attend_core", "ffn_prepare", "ffn_main", "gate_eval", "project_qkv", "project_out",
                                          "moe_plan", "moe_combine", "table_arrange"};
    return (slot >= 0 && slot < KS_COUNT) ? names[slot] : "?";
}

int sentry_profile_read(sentry_ctx* ctx, float* ms, int* launches, int n) {
    if (ctx == nullptr || ms == nullptr || launches == nullptr || n < KS_COUNT)
        return SENTRY_ERR_INVALID_ARG;
    SENTRY_ON_DEVICE(ctx->device);
    SENTRY_CUDA_TRY(cudaDeviceSynchronize());
    for (int i = 0; i < n; ++i) { ms[i] = 0.f; launches[i] = 0; }
    for (ProfRec& r : ctx->prof) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, r.start, r.stop) == cudaSuccess) {
            ms[r.slot] += t;
            launches[r.slot] += 1;
        }
        ctx->pool.push_back(r.start);
        ctx->pool.push_back(r.stop);
    }
    ctx->prof.clear();
    return SENTRY_OK;
}

int sentry_get_last_status(sentry_ctx* ctx, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    SENTRY_ON_DEVICE(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    SENTRY_CUDA_TRY(cudaStreamSynchronize(st));
    unsigned int h = 0;
    SENTRY_CUDA_TRY(cudaMemcpyAsync(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, st));
    SENTRY_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(h), st));
    SENTRY_CUDA_TRY(cudaStreamSynchronize(st));
    return (int)(h & 0x7fffffffu);
}

const char* sentry_status_string(int status) {
    switch (status) {
        case SENTRY_OK: return "ok";
        case SENTRY_ERR_INVALID_ARG: return "invalid argument";
        case SENTRY_ERR_BAD_SHAPE: return "bad shape";
        case SENTRY_ERR_UNSUPPORTED: return "unsupported configuration";
        case SENTRY_ERR_WORKSPACE: return "workspace missing or too small";
        case SENTRY_ERR_CUDA: return "CUDA call failed";
        case SENTRY_ERR_TIMEOUT: return "device wait timed out";
        case SENTRY_ERR_EMPTY_MASK: return "sample with empty modality mask";
        default: return "unknown status";
    }
}

int sentry_num_active_queries(int T_v, int c) { return sentry_num_active(T_v, c); }

size_t sentry_workspace_bytes(const sentry_attend_desc* attend, const sentry_ffn_desc* ffn) {
    size_t need = kMinWorkspace;
    if (attend != nullptr && check_attend_desc(attend) == SENTRY_OK) {
        const size_t a = attend_workspace_bytes(*attend);
        if (a > need) need = a;
    }
    if (ffn != nullptr && check_ffn_desc(ffn) == SENTRY_OK) {
        const size_t f = ffn_workspace_bytes(*ffn);
        if (f > need) need = f;
    }
    return align_up(need, 256);
}

int sentry_set_workspace(sentry_ctx* ctx, void* dev_ptr, size_t bytes) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (dev_ptr != nullptr && !aligned(dev_ptr, 256)) return SENTRY_ERR_INVALID_ARG;
    ctx->workspace = dev_ptr;
    ctx->workspace_bytes = dev_ptr ? bytes : 0;
    return SENTRY_OK;
}

int sentry_selftest_wait_expiry(sentry_ctx* ctx, long long limit_cycles, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > 100000000LL) return SENTRY_ERR_BAD_SHAPE;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_wait_expiry_selftest(ctx, limit_cycles, (cudaStream_t)stream);
}

int sentry_set_option(sentry_ctx* ctx, int option, int value) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    switch (option) {
        case SENTRY_OPT_ATTEND_KERNEL:
            if (value < SENTRY_ATTEND_AUTO || value > SENTRY_ATTEND_TCGEN05) return SENTRY_ERR_INVALID_ARG;
            ctx->attend_kernel = value;
            return SENTRY_OK;
        case SENTRY_OPT_LONG_SELECT:
            if (value < SENTRY_LONG_SELECT_AUTO || value > SENTRY_LONG_SELECT_PER_GROUP) return SENTRY_ERR_INVALID_ARG;
            ctx->long_select = value;
            return SENTRY_OK;
        default:
            return SENTRY_ERR_INVALID_ARG;
    }
}

int sentry_last_launch_count(const sentry_ctx* ctx) { return ctx ? ctx->last_launches : 0; }

int sentry_gate_select(sentry_ctx* ctx, const float* scores, int S, int n_units,
                       const uint32_t* masks, int n_masks, int k, int32_t* kept,
                       uint32_t* kv_groups, int heads_per_group, void* stream) {
    if (ctx == nullptr || scores == nullptr || masks == nullptr || kept == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (!aligned(scores, 4) || !aligned(masks, 4) || !aligned(kept, 4)) return SENTRY_ERR_INVALID_ARG;
    if (S < 1 || n_units < 1 || n_masks < 0 || k < 1 || k > n_units) return SENTRY_ERR_BAD_SHAPE;
    if (n_units > kMaxUnits || S > 65536) return SENTRY_ERR_UNSUPPORTED;
    if (kv_groups != nullptr) {
        if (heads_per_group < 1) return SENTRY_ERR_INVALID_ARG;
        if ((n_units + heads_per_group - 1) / heads_per_group > 32) return SENTRY_ERR_BAD_SHAPE;
    }
    ctx->last_launches = 0;
    if (n_masks == 0) return SENTRY_OK;
    WsAlloc a(ctx->workspace, ctx->workspace_bytes);
    int32_t* rows = a.take<int32_t>((size_t)S * k);
    uint32_t* groups = a.take<uint32_t>((size_t)S);
    if (!a.ok) return SENTRY_ERR_WORKSPACE;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_gate_select(ctx, scores, S, n_units, masks, n_masks, k, kept, kv_groups,
                              heads_per_group, rows, groups, (cudaStream_t)stream);
}

int sentry_gate_select_multi(sentry_ctx* ctx, int S, const sentry_gate_set* sets, int n_sets, void* stream) {
    if (ctx == nullptr || sets == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (n_sets < 1 || n_sets > SENTRY_GATE_MAX_SETS || S < 1) return SENTRY_ERR_BAD_SHAPE;
    if (S > 65536 / SENTRY_GATE_MAX_SETS) return SENTRY_ERR_UNSUPPORTED;
    WsAlloc a(ctx->workspace, ctx->workspace_bytes);
    int32_t* rows[SENTRY_GATE_MAX_SETS];
    uint32_t* groups[SENTRY_GATE_MAX_SETS];
    bool any = false;
    for (int i = 0; i < n_sets; ++i) {
        const sentry_gate_set& g = sets[i];
        if (g.scores == nullptr || g.masks == nullptr || g.kept == nullptr) return SENTRY_ERR_INVALID_ARG;
        if (!aligned(g.scores, 4) || !aligned(g.masks, 4) || !aligned(g.kept, 4)) return SENTRY_ERR_INVALID_ARG;
        if (g.n_units < 1 || g.n_masks < 0 || g.k < 1 || g.k > g.n_units) return SENTRY_ERR_BAD_SHAPE;
        if (g.n_units > kMaxUnits) return SENTRY_ERR_UNSUPPORTED;
        if (g.kv_groups != nullptr) {
            if (g.heads_per_group < 1) return SENTRY_ERR_INVALID_ARG;
            if ((g.n_units + g.heads_per_group - 1) / g.heads_per_group > 32) return SENTRY_ERR_BAD_SHAPE;
        }
        rows[i] = a.take<int32_t>((size_t)S * g.k);
        groups[i] = a.take<uint32_t>((size_t)S);
        any = any || g.n_masks > 0;
    }
    ctx->last_launches = 0;
    if (!any) return SENTRY_OK;
    if (!a.ok) return SENTRY_ERR_WORKSPACE;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_gate_select_multi(ctx, S, sets, n_sets, rows, groups, (cudaStream_t)stream);
}

int sentry_gate_eval(sentry_ctx* ctx, int M, int hidden, int n_layers, const int32_t* layer_offsets,
                     int n_units, const float* zeta, const float* gamma, const float* W1, const float* b1,
                     const float* w2, const float* b2, float* logits, float* gates, void* stream) {
    if (ctx == nullptr || layer_offsets == nullptr || zeta == nullptr || gamma == nullptr || W1 == nullptr ||
        b1 == nullptr || w2 == nullptr || b2 == nullptr || logits == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (M < 1 || M > 16 || hidden < 1 || hidden > 4096 || n_layers < 1 || n_units < 1) return SENTRY_ERR_BAD_SHAPE;
    if (n_units > kMaxUnits) return SENTRY_ERR_UNSUPPORTED;
    ctx->last_launches = 0;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_gate_eval(ctx, zeta, gamma, layer_offsets, n_layers, W1, b1, w2, b2, M, hidden, n_units, logits,
                            gates, (cudaStream_t)stream);
}

int sentry_gate_layer_counts(sentry_ctx* ctx, const int32_t* kept, int n_masks, int k,
                             const int32_t* layer_offsets, int n_layers, int32_t* counts, void* stream) {
    if (ctx == nullptr || kept == nullptr || layer_offsets == nullptr || counts == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (n_masks < 0 || k < 1 || n_layers < 1) return SENTRY_ERR_BAD_SHAPE;
    ctx->last_launches = 0;
    if (n_masks == 0) return SENTRY_OK;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_layer_counts(ctx, kept, n_masks, k, layer_offsets, n_layers, counts, (cudaStream_t)stream);
}

// Body of sentry_attend_fwd and sentry_gate_attend_fwd.  gate_scores != null: the kept heads are
// selected from that table (into kept_heads, which is then an output) instead of being given.
static int attend_body(sentry_ctx* ctx, const sentry_attend_desc* desc, const void* Q,
                       const void* K, const void* V, int32_t* kept_heads,
                       const int32_t* token_modality_ids, const uint32_t* masks,
                       const int32_t* sample_table, const int64_t* sample_offsets,
                       int n_subsets, void* O, int32_t* active_out, const int32_t* active_in,
                       const float* gate_scores, int gate_S, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_attend_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (Q == nullptr || K == nullptr || V == nullptr || O == nullptr || kept_heads == nullptr ||
        token_modality_ids == nullptr || masks == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) ||
        !aligned(kept_heads, 4) || !aligned(token_modality_ids, 4) || !aligned(masks, 4))
        return SENTRY_ERR_INVALID_ARG;
    if (active_in == nullptr && desc->score_mode != 1) {
        if (sample_table == nullptr || sample_offsets == nullptr) return SENTRY_ERR_INVALID_ARG;
        if (n_subsets < 1) return SENTRY_ERR_BAD_SHAPE;
        if (!aligned(sample_table, 4) || !aligned(sample_offsets, 8)) return SENTRY_ERR_INVALID_ARG;
    }
    if (gate_scores != nullptr) {
        if (!aligned(gate_scores, 4)) return SENTRY_ERR_INVALID_ARG;
        if (gate_S < 1) return SENTRY_ERR_BAD_SHAPE;
        if (gate_S > 65536 || desc->Hq > kMaxUnits) return SENTRY_ERR_UNSUPPORTED;
    }
    ctx->last_launches = 0;
    AttendArgs a;
    a.gate_scores = nullptr; a.gate_S = 0; a.kept_out = nullptr;
    a.d = *desc;
    a.Q = Q; a.K = K; a.V = V;
    a.kept_heads = kept_heads;
    a.ids = token_modality_ids;
    a.masks = masks;
    a.sample_table = sample_table;
    a.sample_offsets = sample_offsets;
    a.n_subsets = n_subsets;
    a.O = O;
    a.U_max = sentry_num_active(desc->T, desc->c);
    a.status = ctx->d_status;
    WsAlloc ws(ctx->workspace, ctx->workspace_bytes);
    a.mscore = ws.take<float>((size_t)desc->B * desc->k_h * desc->T);
    int32_t* ws_active = ws.take<int32_t>((size_t)desc->B * desc->k_h * a.U_max);
    if (!ws.ok) return SENTRY_ERR_WORKSPACE;
    a.selection_given = active_in != nullptr;
    a.active = a.selection_given ? const_cast<int32_t*>(active_in)
                                 : (active_out != nullptr ? active_out : ws_active);
    SENTRY_ON_DEVICE(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    a.active_out_user = active_out;
    if (gate_scores != nullptr) {
        // inside the attention launch where that saves a launch worth saving: up to a few waves of
        // CTAs (beyond, the selection repeated in every CTA costs more than one small launch: +5 %
        // on B = 4096)
        const bool inside = ctx->attend_kernel != SENTRY_ATTEND_TCGEN05 &&
                            (attend_bf16_gate_fusable(*desc) || attend_f16_gate_fusable(*desc)) &&
                            (long long)desc->B * desc->Hk <= 8LL * ctx->sm_count;
        if (inside) {   // the fused attention kernel selects the heads itself
            a.gate_scores = gate_scores; a.gate_S = gate_S; a.kept_out = kept_heads;
        } else {        // a gate launch first; its scratch rows are dead before the attention kernels start
            WsAlloc g(ctx->workspace, ctx->workspace_bytes);
            int32_t* rows = g.take<int32_t>((size_t)gate_S * desc->k_h);
            uint32_t* groups = g.take<uint32_t>((size_t)gate_S);
            if (!g.ok) return SENTRY_ERR_WORKSPACE;
            rc = launch_gate_select(ctx, gate_scores, gate_S, desc->Hq, masks, desc->B, desc->k_h, kept_heads, nullptr, 0,
                                    rows, groups, st);
            if (rc != SENTRY_OK) return rc;
        }
    }
    // AUTO takes the kernel that measured faster for the shape: at present the warp-MMA kernels
    // on every shape they support (the tcgen05 kernel is within 10-20 % on T >= 512)
    if (ctx->attend_kernel == SENTRY_ATTEND_TCGEN05 && attend_tc_supported(*desc)) rc = launch_attend_tc(ctx, a, st);
    else rc = attend_bf16_supported(*desc)  ? launch_attend_bf16(ctx, a, st)
              : attend_f16_supported(*desc) ? launch_attend_f16(ctx, a, st)
                                            : launch_attend_generic(ctx, a, st);
    if (rc != SENTRY_OK) return rc;
    if (a.selection_given && active_out != nullptr && active_out != active_in) {
        SENTRY_CUDA_TRY(cudaMemcpyAsync(active_out, active_in,
                                        (size_t)desc->B * desc->k_h * a.U_max * sizeof(int32_t),
                                        cudaMemcpyDeviceToDevice, st));
    }
    return SENTRY_OK;
}

int sentry_attend_fwd(sentry_ctx* ctx, const sentry_attend_desc* desc, const void* Q,
                      const void* K, const void* V, const int32_t* kept_heads,
                      const int32_t* token_modality_ids, const uint32_t* masks,
                      const int32_t* sample_table, const int64_t* sample_offsets,
                      int n_subsets, void* O, int32_t* active_out, const int32_t* active_in,
                      void* stream) {
    return attend_body(ctx, desc, Q, K, V, const_cast<int32_t*>(kept_heads), token_modality_ids, masks, sample_table,
                       sample_offsets, n_subsets, O, active_out, active_in, nullptr, 0, stream);
}

int sentry_gate_attend_fwd(sentry_ctx* ctx, const sentry_attend_desc* desc, const float* head_scores, int S,
                           const void* Q, const void* K, const void* V, const int32_t* token_modality_ids,
                           const uint32_t* masks, const int32_t* sample_table, const int64_t* sample_offsets,
                           int n_subsets, void* O, int32_t* kept_heads_out, int32_t* active_out, void* stream) {
    if (head_scores == nullptr || kept_heads_out == nullptr) return SENTRY_ERR_INVALID_ARG;
    return attend_body(ctx, desc, Q, K, V, kept_heads_out, token_modality_ids, masks, sample_table, sample_offsets,
                       n_subsets, O, active_out, nullptr, head_scores, S, stream);
}

int sentry_sample_table_arrange(sentry_ctx* ctx, int T, int c, const int32_t* token_modality_ids,
                                const int32_t* sample_table, const int64_t* sample_offsets, int n_subsets,
                                int32_t* out_table, void* stream) {
    if (ctx == nullptr || token_modality_ids == nullptr || sample_table == nullptr || sample_offsets == nullptr ||
        out_table == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (!aligned(sample_table, 4) || !aligned(out_table, 4) || !aligned(sample_offsets, 8)) return SENTRY_ERR_INVALID_ARG;
    if (out_table == sample_table) return SENTRY_ERR_INVALID_ARG;
    if (T < 1 || c < 1 || n_subsets < 1) return SENTRY_ERR_BAD_SHAPE;
    if (T > 32768 || n_subsets > 65536) return SENTRY_ERR_UNSUPPORTED;
    ctx->last_launches = 0;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_table_arrange(ctx, token_modality_ids, T, c, sample_table, sample_offsets, n_subsets, out_table,
                                (cudaStream_t)stream);
}

int sentry_ffn_fwd(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* X, const void* W1,
                   const void* W2, const int32_t* kept_channels, const int32_t* list_of_sample,
                   const int32_t* token_modality_ids, const uint32_t* masks, void* Y,
                   void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_ffn_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (X == nullptr || W1 == nullptr || W2 == nullptr || Y == nullptr || kept_channels == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if ((token_modality_ids == nullptr) != (masks == nullptr)) return SENTRY_ERR_INVALID_ARG;
    if (desc->n_lists > 1 && list_of_sample == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(W1, 16) || !aligned(W2, 16) || !aligned(Y, 16) ||
        !aligned(kept_channels, 4))
        return SENTRY_ERR_INVALID_ARG;
    ctx->last_launches = 0;
    FfnArgs a = {};
    a.d = *desc;
    a.X = X; a.W1 = W1; a.W2 = W2;
    a.kept = kept_channels;
    a.list_of_sample = list_of_sample;
    a.ids = token_modality_ids;
    a.masks = masks;
    a.Y = Y;
    a.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_ffn(ctx, a, ctx->workspace, ctx->workspace_bytes, nullptr, (cudaStream_t)stream);
}

static int check_proj_desc(const sentry_proj_desc* d) {
    if (d == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (d->dtype != SENTRY_F32 && d->dtype != SENTRY_BF16 && d->dtype != SENTRY_F16) return SENTRY_ERR_INVALID_ARG;
    if (d->B < 1 || d->T < 1 || d->D < 1 || d->Hq < 1 || d->Hk < 1 || d->d < 1 || d->k_h < 1) return SENTRY_ERR_BAD_SHAPE;
    if (d->Hq % d->Hk != 0 || d->k_h > d->Hq) return SENTRY_ERR_BAD_SHAPE;
    if (d->Hk > 32 || d->k_h > 64 || d->D > 8192 || d->k_h * d->d > 8192) return SENTRY_ERR_UNSUPPORTED;
    if ((long long)d->B * d->T > 0x7fffffffLL) return SENTRY_ERR_UNSUPPORTED;
    return SENTRY_OK;
}

int sentry_project_qkv(sentry_ctx* ctx, const sentry_proj_desc* desc, const void* X, const void* WQ,
                       const void* WK, const void* WV, const int32_t* kept_heads,
                       const int32_t* token_modality_ids, const uint32_t* masks, void* Q, void* K, void* V,
                       void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_proj_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (X == nullptr || WQ == nullptr || WK == nullptr || WV == nullptr || kept_heads == nullptr ||
        token_modality_ids == nullptr || masks == nullptr || Q == nullptr || K == nullptr || V == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(WQ, 16) || !aligned(WK, 16) || !aligned(WV, 16) || !aligned(Q, 16) ||
        !aligned(K, 16) || !aligned(V, 16))
        return SENTRY_ERR_INVALID_ARG;
    ctx->last_launches = 0;
    ProjArgs a = {};
    a.d = *desc;
    a.X = X; a.WQ = WQ; a.WK = WK; a.WV = WV;
    a.kept_heads = kept_heads; a.ids = token_modality_ids; a.masks = masks;
    a.Q = Q; a.K = K; a.V = V;
    a.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    if (project_qkv_tc_f16_supported(*desc)) return launch_project_qkv_tc_f16(ctx, a, (cudaStream_t)stream);
    return project_qkv_tc_supported(*desc) ? launch_project_qkv_tc(ctx, a, (cudaStream_t)stream)
                                           : launch_project_qkv_generic(ctx, a, (cudaStream_t)stream);
}

int sentry_project_out(sentry_ctx* ctx, const sentry_proj_desc* desc, const void* A, const void* WO,
                       const int32_t* kept_heads, const int32_t* token_modality_ids, const uint32_t* masks,
                       void* out, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_proj_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (A == nullptr || WO == nullptr || kept_heads == nullptr || token_modality_ids == nullptr || masks == nullptr ||
        out == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (!aligned(A, 16) || !aligned(WO, 16) || !aligned(out, 16)) return SENTRY_ERR_INVALID_ARG;
    ctx->last_launches = 0;
    ProjArgs a = {};
    a.d = *desc;
    a.A = A; a.WO = WO;
    a.kept_heads = kept_heads; a.ids = token_modality_ids; a.masks = masks;
    a.out = out;
    a.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    if (project_out_tc_f16_supported(*desc)) return launch_project_out_tc_f16(ctx, a, (cudaStream_t)stream);
    return project_out_tc_supported(*desc) ? launch_project_out_tc(ctx, a, (cudaStream_t)stream)
                                           : launch_project_out_generic(ctx, a, (cudaStream_t)stream);
}

static int check_moe_desc(const sentry_moe_desc* d) {
    if (d == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (d->dtype != SENTRY_F32 && d->dtype != SENTRY_BF16 && d->dtype != SENTRY_F16) return SENTRY_ERR_INVALID_ARG;
    if (d->N < 1 || d->D < 1 || d->F < 1 || d->E < 1 || d->top_k < 1 || d->k_c < 1) return SENTRY_ERR_BAD_SHAPE;
    if (d->k_c > d->F) return SENTRY_ERR_BAD_SHAPE;
    if (d->D % 8 != 0 || d->D > 1024 || d->E > 4096 || d->top_k > 64) return SENTRY_ERR_UNSUPPORTED;
    if ((long long)d->N * d->top_k > 0x7fffffffLL - 8192) return SENTRY_ERR_UNSUPPORTED;
    return SENTRY_OK;
}

size_t sentry_moe_workspace_bytes(const sentry_moe_desc* desc) {
    return check_moe_desc(desc) == SENTRY_OK ? align_up(moe_workspace_bytes(*desc), 256) : 0;
}

size_t sentry_moe_packed_bytes(const sentry_moe_desc* desc) {
    return check_moe_desc(desc) == SENTRY_OK ? moe_packed_bytes(*desc) : 0;
}

int sentry_moe_prepack(sentry_ctx* ctx, const sentry_moe_desc* desc, const void* W1, const void* W2,
                       const int32_t* kept_channels, void* packed, size_t packed_bytes, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_moe_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (W1 == nullptr || W2 == nullptr || kept_channels == nullptr || packed == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (!aligned(W1, 16) || !aligned(W2, 16) || !aligned(kept_channels, 4) || !aligned(packed, 256))
        return SENTRY_ERR_INVALID_ARG;
    if (packed_bytes < moe_packed_bytes(*desc)) return SENTRY_ERR_WORKSPACE;
    ctx->last_launches = 0;
    MoeArgs m = {};
    m.d = *desc;
    m.W1 = W1; m.W2 = W2;
    m.kept = kept_channels;
    m.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_moe_prepack(ctx, m, packed, (cudaStream_t)stream);
}

int sentry_moe_ffn_fwd(sentry_ctx* ctx, const sentry_moe_desc* desc, const void* X, const void* W1,
                       const void* W2, const int32_t* kept_channels, const void* packed,
                       const int32_t* expert_ids, const float* expert_weights, void* Y, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_moe_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (X == nullptr || Y == nullptr || expert_ids == nullptr || expert_weights == nullptr)
        return SENTRY_ERR_INVALID_ARG;
    if (packed == nullptr && (W1 == nullptr || W2 == nullptr || kept_channels == nullptr))
        return SENTRY_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(Y, 16) || !aligned(expert_ids, 4) || !aligned(expert_weights, 4))
        return SENTRY_ERR_INVALID_ARG;
    if (packed != nullptr ? !aligned(packed, 256) : (!aligned(W1, 16) || !aligned(W2, 16) || !aligned(kept_channels, 4)))
        return SENTRY_ERR_INVALID_ARG;
    ctx->last_launches = 0;
    MoeArgs m = {};
    m.d = *desc;
    m.X = X; m.W1 = W1; m.W2 = W2;
    m.kept = kept_channels;
    m.expert_ids = expert_ids;
    m.expert_weights = expert_weights;
    m.Y = Y;
    m.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_moe_ffn(ctx, m, ctx->workspace, ctx->workspace_bytes, packed, (cudaStream_t)stream);
}

size_t sentry_ffn_packed_bytes(const sentry_ffn_desc* desc) {
    return check_ffn_desc(desc, true) == SENTRY_OK ? ffn_packed_bytes(*desc) : 0;
}

int sentry_ffn_prepack(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* W1, const void* W2,
                       const int32_t* kept_channels, void* packed, size_t packed_bytes, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_ffn_desc(desc, true);
    if (rc == SENTRY_OK && desc->dtype == SENTRY_FP8_E4M3 && !ffn_tc_fp8_supported(*desc)) rc = SENTRY_ERR_UNSUPPORTED;
    if (rc != SENTRY_OK) return rc;
    if (W1 == nullptr || W2 == nullptr || kept_channels == nullptr || packed == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (!aligned(W1, 16) || !aligned(W2, 16) || !aligned(kept_channels, 4) || !aligned(packed, 256))
        return SENTRY_ERR_INVALID_ARG;
    if (packed_bytes < ffn_packed_bytes(*desc)) return SENTRY_ERR_WORKSPACE;
    ctx->last_launches = 0;
    FfnArgs a = {};
    a.d = *desc;
    a.W1 = W1; a.W2 = W2;
    a.kept = kept_channels;
    a.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_ffn_prepack(ctx, a, packed, (cudaStream_t)stream);
}

int sentry_ffn_fwd_fp8(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* X_e4m3, const void* packed,
                       const int32_t* list_of_sample, const int32_t* token_modality_ids, const uint32_t* masks,
                       float scale_x, float scale_w1, float scale_w2, float scale_h, void* Y_bf16, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_ffn_desc(desc, true);
    if (rc != SENTRY_OK) return rc;
    if (desc->dtype != SENTRY_FP8_E4M3) return SENTRY_ERR_INVALID_ARG;
    if (!ffn_tc_fp8_supported(*desc)) return SENTRY_ERR_UNSUPPORTED;
    if (X_e4m3 == nullptr || packed == nullptr || Y_bf16 == nullptr) return SENTRY_ERR_INVALID_ARG;
    if ((token_modality_ids == nullptr) != (masks == nullptr)) return SENTRY_ERR_INVALID_ARG;
    if (desc->n_lists > 1 && list_of_sample == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (!aligned(X_e4m3, 16) || !aligned(Y_bf16, 16) || !aligned(packed, 256)) return SENTRY_ERR_INVALID_ARG;
    if (!(scale_x > 0.f) || !(scale_w1 > 0.f) || !(scale_w2 > 0.f) || !(scale_h > 0.f)) return SENTRY_ERR_INVALID_ARG;
    ctx->last_launches = 0;
    FfnArgs a = {};
    a.d = *desc;
    a.X = X_e4m3;
    a.list_of_sample = list_of_sample;
    a.ids = token_modality_ids;
    a.masks = masks;
    a.Y = Y_bf16;
    a.status = ctx->d_status;
    a.fp8_a_scale = scale_x * scale_w1;
    a.fp8_h_inv = 1.0f / scale_h;
    a.fp8_y_scale = scale_h * scale_w2;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_ffn(ctx, a, ctx->workspace, ctx->workspace_bytes, packed, (cudaStream_t)stream);
}

int sentry_ffn_prepack_fp8(sentry_ctx* ctx, const sentry_ffn_desc* desc, const uint8_t* W1_e4m3, const uint8_t* W2_e4m3,
                           float scale_w1, float scale_w2, const int32_t* kept_channels, void* packed,
                           size_t packed_bytes, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_ffn_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (W1_e4m3 == nullptr || W2_e4m3 == nullptr || kept_channels == nullptr || packed == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (!aligned(kept_channels, 4) || !aligned(packed, 256)) return SENTRY_ERR_INVALID_ARG;
    if (!(scale_w1 == scale_w1) || !(scale_w2 == scale_w2)) return SENTRY_ERR_INVALID_ARG;   // NaN scales
    if (packed_bytes < ffn_packed_bytes(*desc)) return SENTRY_ERR_WORKSPACE;
    ctx->last_launches = 0;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_ffn_prepack_fp8(ctx, *desc, W1_e4m3, W2_e4m3, scale_w1, scale_w2, kept_channels, packed,
                                  (cudaStream_t)stream);
}

int sentry_ffn_fwd_packed(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* X, const void* packed,
                          const int32_t* list_of_sample, const int32_t* token_modality_ids,
                          const uint32_t* masks, void* Y, void* stream) {
    if (ctx == nullptr) return SENTRY_ERR_INVALID_ARG;
    int rc = check_ffn_desc(desc);
    if (rc != SENTRY_OK) return rc;
    if (X == nullptr || packed == nullptr || Y == nullptr) return SENTRY_ERR_INVALID_ARG;
    if ((token_modality_ids == nullptr) != (masks == nullptr)) return SENTRY_ERR_INVALID_ARG;
    if (desc->n_lists > 1 && list_of_sample == nullptr) return SENTRY_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(Y, 16) || !aligned(packed, 256)) return SENTRY_ERR_INVALID_ARG;
    ctx->last_launches = 0;
    FfnArgs a = {};
    a.d = *desc;
    a.X = X;
    a.list_of_sample = list_of_sample;
    a.ids = token_modality_ids;
    a.masks = masks;
    a.Y = Y;
    a.status = ctx->d_status;
    SENTRY_ON_DEVICE(ctx->device);
    return launch_ffn(ctx, a, ctx->workspace, ctx->workspace_bytes, packed, (cudaStream_t)stream);
}

}  // extern "C"

/*
 * sentry.h -- C ABI of libsentry: inference through a deployment-pruned
 * multimodal transformer layer on one NVIDIA B200 (sm_100a).
 *
 * Three operations, in the order a pruned layer uses them:
 *   sentry_gate_select  modality-conditioned selection of the attention heads
 *                       and FFN channels to keep         (SentryGate, Sec. 4.6)
 *   sentry_attend_fwd   sparse grouped-query attention over the kept heads
 *                       (SentryAttend, Sec. 4.4, Eq. 6)
 *   sentry_ffn_fwd      feed-forward block over the kept channels only
 *                       (Sec. 4.6: W1' = W1[:, N_keep], W2' = W2[N_keep, :])
 *
 * Conventions
 *   - Every tensor argument is a caller-owned DEVICE pointer unless it says
 *     "host".  The library never allocates or frees tensors; scratch comes
 *     from a caller-provided workspace (sentry_set_workspace).
 *   - All calls enqueue work on the CUDA stream passed as `stream`
 *     (a cudaStream_t cast to void*, NULL = default stream) and return without
 *     synchronising.  Calls that share a context and its workspace must be
 *     ordered on one stream (or otherwise not overlap).
 *   - Return value: 0 = SENTRY_OK, negative = error found on the host BEFORE any
 *     launch (nothing was enqueued).  Conditions only the device can see (a
 *     sample with an empty modality mask, a bounded wait that ran out) are
 *     OR-ed into a device status word, read with sentry_get_last_status.
 *   - Dense tensors are contiguous row-major in the shapes given; base
 *     pointers must be 16-byte aligned.
 *   - Modality masks: bit j of a mask = modality j is present.  A score table
 *     has one row per mask value (row index = the mask's bit pattern).
 *   - There is no CPU fallback: without a CUDA device every compute call fails.
 */
#ifndef SENTRY_H
#define SENTRY_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SENTRY_API __attribute__((visibility("default")))
#else
#define SENTRY_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sentry_ctx sentry_ctx; /* opaque: device, workspace, status word */

typedef enum {
    SENTRY_OK = 0,
    SENTRY_ERR_INVALID_ARG = -1, /* null pointer, bad enum, misaligned pointer */
    SENTRY_ERR_BAD_SHAPE = -2,   /* dimension out of range or inconsistent */
    SENTRY_ERR_UNSUPPORTED = -3, /* valid but not implemented on this path */
    SENTRY_ERR_WORKSPACE = -4,   /* workspace missing or too small */
    SENTRY_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed */
    SENTRY_ERR_TIMEOUT = -6,     /* device: a bounded wait expired (status word) */
    SENTRY_ERR_EMPTY_MASK = -7   /* device: a sample had no modality present */
} sentry_status;

/* bits of the device status word returned by sentry_get_last_status */
#define SENTRY_STATUS_BIT_TIMEOUT 1u
#define SENTRY_STATUS_BIT_EMPTY_MASK 2u
#define SENTRY_STATUS_BIT_BAD_INDEX 4u /* a kept index / token id out of range was skipped */

/* SENTRY_F16 (IEEE half; the FP16 post-training-quantisation point of Sec. 5): taken by every entry point.  The
 * FFN pair and the Sparse-MoE block run on tcgen05 with fp16 operands, attention on the warp-MMA kernels with fp16
 * operands (the tcgen05 attention kernel is bf16 only), the projections on tcgen05 with fp16 operands. */
typedef enum { SENTRY_F32 = 0, SENTRY_BF16 = 1, SENTRY_F16 = 2, SENTRY_FP8_E4M3 = 3 /* FFN only, see sentry_ffn_fwd_fp8 */ } sentry_dtype;

/* Create / destroy a context bound to CUDA device `device`.  Creation
 * allocates one small device status word; nothing else. */
SENTRY_API int sentry_create(sentry_ctx** out, int device);
SENTRY_API int sentry_destroy(sentry_ctx* ctx);

/* Synchronise `stream`, return the device status word (>= 0, SENTRY_STATUS_BIT_*)
 * and clear it; negative on CUDA failure. */
SENTRY_API int sentry_get_last_status(sentry_ctx* ctx, void* stream);

SENTRY_API const char* sentry_status_string(int status);

/* U(T_v) = max(1, min(T_v, c * ceil(ln T_v))): how many queries per head stay
 * active among T_v present tokens (Sec. 4.4; the paper's example T=128, c=5
 * gives 25).  It is also the number of sampled keys per query, i.e. the width
 * of a sample-table row.  Host function, no device work.  Returns 0 for T_v<=0. */
SENTRY_API int sentry_num_active_queries(int T_v, int c);

/* Scratch memory.  sentry_workspace_bytes returns an upper bound for any
 * sequence of the three calls with the given descriptors (either may be NULL);
 * sentry_set_workspace hands the library a device buffer of at least that many
 * bytes, 256-byte aligned, which it uses until replaced.  The caller keeps
 * ownership. */
struct sentry_attend_desc;
struct sentry_ffn_desc;
SENTRY_API size_t sentry_workspace_bytes(const struct sentry_attend_desc* attend,
                              const struct sentry_ffn_desc* ffn);
SENTRY_API int sentry_set_workspace(sentry_ctx* ctx, void* dev_ptr, size_t bytes);

/* ---------------------------------------------------------------------------
 * SentryGate selection (Sec. 4.6 "Applying SentryGate": gate outputs under a
 * fixed modality mask are thresholded by a pruning ratio; here the ratio is an
 * integer budget k per unit type).
 *
 *   scores  [S, n_units] fp32, row s = gate outputs under mask value s
 *   masks   [n_masks] u32, each < S (a mask >= S is skipped and flagged BAD_INDEX)
 *   k       budget, 1 <= k <= n_units
 *   kept    out [n_masks, k] i32: the k units with the highest score in row
 *           masks[i]; equal scores -> the lower index wins (+0 == -0; NaN ranks
 *           below every number); written in ASCENDING index order
 *   kv_groups  out [n_masks] u32 or NULL: bit g set iff some kept unit maps to
 *           KV group g = floor(unit / heads_per_group) ("head pruning with GQA
 *           consistency"); needs heads_per_group >= 1 and n_units/heads_per_group <= 32
 * Needs a workspace of S*k*4 bytes.
 */
SENTRY_API int sentry_gate_select(sentry_ctx* ctx, const float* scores, int S, int n_units,
                       const uint32_t* masks, int n_masks, int k, int32_t* kept,
                       uint32_t* kv_groups, int heads_per_group, void* stream);

/* Several selections over the same S mask values in ONE launch (the heads and
 * the channels of a layer, or the units of several layers): every member of
 * `sets` (host array, 1 <= n_sets <= SENTRY_GATE_MAX_SETS) has the meaning of
 * the like-named sentry_gate_select arguments, and the result of each set is
 * what sentry_gate_select would write for it.  A set with n_masks * k > 16384
 * needs one more launch for its fan-out.  Workspace: the sum over the sets of
 * S*k*4 + S*4 bytes, each rounded up to 256. */
#define SENTRY_GATE_MAX_SETS 4
typedef struct sentry_gate_set {
    const float* scores;   /* [S, n_units] fp32 */
    int n_units, k;
    const uint32_t* masks; /* [n_masks] u32 */
    int n_masks;
    int32_t* kept;         /* out [n_masks, k] */
    uint32_t* kv_groups;   /* out [n_masks] or NULL */
    int heads_per_group;
} sentry_gate_set;
SENTRY_API int sentry_gate_select_multi(sentry_ctx* ctx, int S, const sentry_gate_set* sets, int n_sets,
                             void* stream);

/* ---------------------------------------------------------------------------
 * SentryGate on the device (Sec. 4.2, Eq. 1) and the cross-layer threshold of
 * Sec. 4.6 (the gate outputs of all layers are ranked together and cut by one
 * threshold that the pruning ratio fixes).
 *
 * Units of all layers are concatenated: layer l owns the unit indices
 * [layer_offsets[l], layer_offsets[l+1]), layer_offsets[n_layers] = n_units.
 *   z_i(s) = zeta[i] + gamma[l(i)] * f_i(m_s),   g_i(s) = 1 / (1 + exp(-z_i(s)))
 *   f_i(m) = w2[i,:] . relu(W1[i,:,:] m + b1[i,:]) + b2[i]
 * with m_s in {0,1}^M the bits of the mask value s (bit j = modality j present).
 * The paper says "a two-layer MLP with a nonlinearity"; ReLU is this library's
 * reading.  All parameters fp32, device:
 *   zeta [n_units], gamma [n_layers], W1 [n_units, hidden, M], b1, w2 [n_units, hidden], b2 [n_units]
 *   logits out [2^M, n_units] (row index = mask value): the score table for
 *          sentry_gate_select -- ranking z equals ranking g and does not saturate
 *   gates  out [2^M, n_units] or NULL: g itself
 * The global threshold is then sentry_gate_select(logits, S = 2^M, n_units,
 * masks, k = units kept over ALL layers); sentry_gate_layer_counts turns the
 * kept lists [n_masks, k] (ascending) into counts [n_masks, n_layers] per layer
 * (the kept units of layer l are the next counts[l] entries of the list).
 */
SENTRY_API int sentry_gate_eval(sentry_ctx* ctx, int M, int hidden, int n_layers,
                     const int32_t* layer_offsets, int n_units, const float* zeta,
                     const float* gamma, const float* W1, const float* b1, const float* w2,
                     const float* b2, float* logits, float* gates, void* stream);
SENTRY_API int sentry_gate_layer_counts(sentry_ctx* ctx, const int32_t* kept, int n_masks, int k,
                             const int32_t* layer_offsets, int n_layers, int32_t* counts,
                             void* stream);

/* ---------------------------------------------------------------------------
 * Gate selection for callers that cannot allocate device memory.
 *
 * (No counterpart in the paper: this is a deployment convenience, not part of
 * the method.)  Some hosts of this library may not call cudaMalloc at all --
 * a plug-in that lives inside another runtime's memory pool, or a service
 * that pins its device-memory budget at start-up and forbids growth.  They
 * cannot create a context (sentry_create allocates a status word) nor hand
 * over a workspace.  This entry point needs neither: the per-score-row
 * scratch of the selection sits in a fixed array inside the library image,
 * SENTRY_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the
 * process exits.  It calls no cudaMalloc/cudaFree and no allocating routine.
 *
 * Arguments and results are those of sentry_gate_select, with `device` in
 * place of the context, plus
 *   status  device pointer to one u32 or NULL: SENTRY_STATUS_BIT_* flags are
 *           OR-ed into it (the caller clears it).  With NULL the flags go to an
 *           internal word that nothing reads.
 * Limits: n_units <= 12288, and 256 + roundup256(S*k*4) + S*4 <=
 * SENTRY_STATIC_SCRATCH_BYTES, else SENTRY_ERR_UNSUPPORTED / SENTRY_ERR_WORKSPACE
 * before anything is enqueued.
 * The first call on a device looks up the array's device address (one runtime
 * query, cached); make that first call before any stream capture begins.
 * All calls on a device share the one array and it keeps the previous call's
 * contents (the library clears the word that must start at zero): calls whose
 * kernels could overlap on the GPU -- different streams without an ordering
 * between them -- race.  Order them on one stream or with events.
 */
#define SENTRY_STATIC_SCRATCH_BYTES (256 * 1024)
SENTRY_API int sentry_gate_select_static(int device, const float* scores, int S, int n_units,
                              const uint32_t* masks, int n_masks, int k, int32_t* kept,
                              uint32_t* kv_groups, int heads_per_group, uint32_t* status,
                              void* stream);

/* ---------------------------------------------------------------------------
 * SentryAttend forward (Sec. 4.4, Eq. 6) on the kept heads of every sample.
 *
 * Per sample b, with present tokens = { t : bit ids[t] of masks[b] is set }
 * (T_v of them, U = sentry_num_active_queries(T_v, c)), and per kept head h
 * with KV group g = floor(h / (Hq/Hk)):
 *   1. sparsity score of each present query i over its sampled keys S_i:
 *        M_i = max_{j in S_i} s_ij - mean_{j in S_i} s_ij,  s_ij = q_i.k_j/sqrt(d)
 *   2. the U present queries with the largest M_i are active (ties -> lower index)
 *   3. active rows:   O[i] = softmax_j(s_ij) V_g[j] over ALL present keys j (Eq. 6)
 *   4. other present rows: O[i] = mean over present keys of V_g[j]
 *   5. rows of absent-modality tokens: 0.   Pruned heads are not computed.
 */
typedef struct sentry_attend_desc {
    int B, T, Hq, Hk, d; /* batch, tokens per sample, query heads, KV heads, head dim */
    int k_h;             /* kept heads per sample (same for every sample) */
    int dtype;           /* sentry_dtype of Q, K, V, O */
    int c;               /* sparsity constant of U = c*ceil(ln T_v); the paper uses 5 */
    int score_mode;      /* 0: S_i from the sample table; 1: S_i = all present keys;
                            2: as 0, the table of every subset stored entry-major */
} sentry_attend_desc;

/*   Q [B,Hq,T,d]; K, V [B,Hk,T,d]; O out [B,k_h,T,d] (heads in kept-list order)
 *   kept_heads [B,k_h] i32 ascending, in [0,Hq)
 *   token_modality_ids [T] i32 in [0,32); masks [B] u32
 *   sample_table i32 + sample_offsets i64 [2^M entries, indexed by mask value]
 *     (score_mode 0 and 2, else NULL): sample_table + sample_offsets[m] is the
 *     [T_v, U] table of the subset m; row i = the U key positions (indices into
 *     the present-token list, each in [0,T_v)) on which query position i is scored.
 *     Subsets with equal T_v may share one table.  n_subsets = entries of sample_offsets.
 *     score_mode 2: the same numbers stored [U, T_v] (sample j of query position i
 *     at j*T_v + i), so that the queries of a warp read one sample with one
 *     128-byte access; the result is bit for bit that of score_mode 0.
 *   active_out [B,k_h,U_max] i32 or NULL, U_max = sentry_num_active_queries(T,c):
 *     the active token indices, ascending, padded with -1
 *   active_in  same shape or NULL: if given, step 1-2 are skipped and these
 *     rows are the active ones (explicit-selection mode)
 * Supported: d in {16,32,64}; Hq % Hk == 0; T <= 32768.  Workspace: see
 * sentry_workspace_bytes.
 */
SENTRY_API int sentry_attend_fwd(sentry_ctx* ctx, const sentry_attend_desc* desc, const void* Q,
                      const void* K, const void* V, const int32_t* kept_heads,
                      const int32_t* token_modality_ids, const uint32_t* masks,
                      const int32_t* sample_table, const int64_t* sample_offsets,
                      int n_subsets, void* O, int32_t* active_out,
                      const int32_t* active_in, void* stream);

/* SentryGate's head selection and SentryAttend in one call: the kept heads of
 * every sample are the k_h best of row masks[b] of head_scores [S, Hq] fp32
 * (the rule of sentry_gate_select: score descending, equal scores -> lower
 * index, NaN below every number; ascending output) and attention runs on them.
 * kept_heads_out [B,k_h] i32 receives the lists (O's head axis follows them).
 * Where K and V of a group fit in shared memory (bf16, Hq <= 64) and the batch
 * is at most a few waves of CTAs (B*Hk <= 8 x the SM count) the attention
 * kernel selects the heads itself -- one launch instead of two, which is what
 * the short workloads' step time is made of; otherwise this is
 * sentry_gate_select followed by sentry_attend_fwd.  A mask >= S is flagged
 * BAD_INDEX (the one-launch form then uses row 0 for that sample, the
 * two-launch form leaves its list unwritten).  No forced selection here.
 * Workspace: what sentry_attend_fwd needs for the descriptor, and at least
 * S*k_h*4 + S*4 + 512 bytes (the two-launch form's gate rows). */
SENTRY_API int sentry_gate_attend_fwd(sentry_ctx* ctx, const sentry_attend_desc* desc,
                           const float* head_scores, int S, const void* Q, const void* K,
                           const void* V, const int32_t* token_modality_ids,
                           const uint32_t* masks, const int32_t* sample_table,
                           const int64_t* sample_offsets, int n_subsets, void* O,
                           int32_t* kept_heads_out, int32_t* active_out, void* stream);

/* Preparation of the sample tables for score_mode 2, once per set of tables
 * (Sec. 4.4 fixes WHICH keys a query is scored on, not the order they are
 * visited in).  Reads the tables as score_mode 0 takes them ([T_v, U] per
 * subset, offsets per mask value) and writes them entry-major into out_table
 * (same size, same offsets, must not overlap sample_table), the U members of
 * every query's set reordered so that the 8 queries of a shared-memory access
 * phase read key rows on different banks wherever the sets allow it.  The sets
 * themselves are unchanged; the sparsity scores change by the rounding of a
 * different summation order only.  Subsets sharing one table are written
 * twice with the same values.  Entries outside [0,T_v) are flagged BAD_INDEX
 * and replaced by 0.  U(T, c) <= 64.  Where it pays: the kernels that keep a
 * group's K rows in shared memory for the whole call (about -3 % on them:
 * conflicts are a quarter of what they were, the gather is latency-bound
 * otherwise).  Sequences long enough for K to be walked in segments are better
 * served by the plain transposition of ascending tables, which keeps a warp's
 * samples of one step in one segment. */
SENTRY_API int sentry_sample_table_arrange(sentry_ctx* ctx, int T, int c,
                                const int32_t* token_modality_ids, const int32_t* sample_table,
                                const int64_t* sample_offsets, int n_subsets,
                                int32_t* out_table, void* stream);

/* The same with the pruned weights materialised ONCE, as Sec. 4.6 describes
 * ("materialize a pruned model" per modality mask and budget), instead of on
 * every call:
 *   sentry_ffn_packed_bytes   size of the buffer for W1' and W2' of all lists
 *                             (0 for an invalid descriptor; only D, F, k_c,
 *                             n_lists and dtype matter)
 *   sentry_ffn_prepack        gathers W1[:, N] and W2[N, :] of every list into
 *                             `packed` (caller-owned device buffer of at least
 *                             that size, 256-byte aligned; the layout is the
 *                             library's own)
 *   sentry_ffn_fwd_packed     sentry_ffn_fwd with `packed` in place of W1, W2 and
 *                             kept_channels; the descriptor must have the same
 *                             D, F, k_c, n_lists and dtype as at prepack time.
 * The buffer stays valid until the weights or the kept lists change. */
SENTRY_API size_t sentry_ffn_packed_bytes(const sentry_ffn_desc* desc);
SENTRY_API int sentry_ffn_prepack(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* W1,
                       const void* W2, const int32_t* kept_channels, void* packed,
                       size_t packed_bytes, void* stream);
/* The weights kept in FP8 (Sec. 5: the FP8 point of the quantisation axis is the one that pays in STORAGE): W1 [D,F]
 * and W2 [F,D] as e4m3 codes (one byte each: sign, 4 exponent bits with bias 7, 3 fraction bits, no infinities), each
 * with one fp32 scale; an element is decode(code) * scale.  sentry_ffn_prepack_fp8 materialises W1[:, N], W2[N, :]
 * of every list from them into `packed`, rounded once to desc->dtype, in the layout sentry_ffn_fwd_packed reads: the
 * FFN then runs as for 16-bit weights (the arithmetic is not FP8: weights-only quantisation). */
SENTRY_API int sentry_ffn_prepack_fp8(sentry_ctx* ctx, const sentry_ffn_desc* desc, const uint8_t* W1_e4m3,
                           const uint8_t* W2_e4m3, float scale_w1, float scale_w2,
                           const int32_t* kept_channels, void* packed, size_t packed_bytes, void* stream);
/* FP8 ARITHMETIC (Sec. 5, the FP8 point taken to the tensor cores; desc->dtype = SENTRY_FP8_E4M3, D = 128, 256 or 384):
 * X [B,T,D] and the weights are e4m3 codes with per-tensor scales scale_x, scale_w1, scale_w2; the hidden
 * activations are requantised to e4m3 with scale_h (a calibration constant of the caller); Y is bf16:
 *   z = (x_q . W1_q[:, N]) * (scale_x*scale_w1);  h_q = e4m3(gelu(z) / scale_h)   (nearest, saturating at 448)
 *   y = (h_q . W2_q[N, :]) * (scale_h*scale_w2)
 * with exact e4m3 x e4m3 products accumulated in fp32 (tcgen05 kind::f8f6f4).  The weights come from
 * sentry_ffn_prepack called with the same FP8 descriptor on the e4m3 W1 [D,F], W2 [F,D] (it gathers bytes).
 * All scales > 0.  Other shapes: SENTRY_ERR_UNSUPPORTED. */
SENTRY_API int sentry_ffn_fwd_fp8(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* X_e4m3,
                       const void* packed, const int32_t* list_of_sample,
                       const int32_t* token_modality_ids, const uint32_t* masks, float scale_x,
                       float scale_w1, float scale_w2, float scale_h, void* Y_bf16, void* stream);
SENTRY_API int sentry_ffn_fwd_packed(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* X,
                          const void* packed, const int32_t* list_of_sample,
                          const int32_t* token_modality_ids, const uint32_t* masks, void* Y,
                          void* stream);

/* ---------------------------------------------------------------------------
 * Sparse-MoE block with expert-internal channel pruning (Sec. 4.6, "Extending
 * SentryGate to Sparse-MoE Architectures": the number of experts and the top-k
 * routing rule stay as they are; every expert e keeps its own channel set N_e
 * of its own FFN, W1_e' = W1_e[:, N_e], W2_e' = W2_e[N_e, :]).  The routing
 * result is an input.  For every token t
 *   y_t = sum_j w[t,j] * ( gelu(x_t . W1_e[:, N_e]) . W2_e[N_e, :] ),  e = expert_ids[t,j],
 * gelu as in sentry_ffn_fwd; the sum runs over the slots j = 0..top_k-1 in
 * that order, accumulated in fp32 (each term first rounded to `dtype`).
 *
 *   X [N,D]; W1 [E,D,F]; W2 [E,F,D] (row-major, dtype); kept_channels [E,k_c] i32
 *   expert_ids [N,top_k] i32: -1 = slot not routed (contributes nothing); any
 *     other value outside [0,E) is skipped and flagged BAD_INDEX
 *   expert_weights [N,top_k] fp32 (whatever the router produced; not renormalised)
 *   Y out [N,D] dtype; a token with no routed slot gets zeros
 * All device pointers, 16-byte aligned; D % 8 == 0, D <= 1024, E <= 4096,
 * N*top_k < 2^31.  bf16 with D in {128,256,384} runs on the tcgen05 kernel of
 * sentry_ffn_fwd with one weight set per expert; other shapes on the plain
 * ALUs.  Scratch (row plan, per-slot results, and W1', W2' unless `packed` is
 * given) comes from the workspace: sentry_moe_workspace_bytes.
 *
 *   sentry_moe_packed_bytes / sentry_moe_prepack: materialise W1_e', W2_e' of
 *     all experts once (same contract as sentry_ffn_prepack)
 *   sentry_moe_ffn_fwd: `packed` NULL -> W1, W2, kept_channels are gathered on
 *     every call; otherwise they are ignored (may be NULL) and `packed` is used.
 */
typedef struct sentry_moe_desc {
    int N;      /* tokens */
    int D, F;   /* d_model, d_ff of one expert */
    int E;      /* experts */
    int top_k;  /* routing slots per token */
    int k_c;    /* kept channels per expert */
    int dtype;  /* sentry_dtype of X, W1, W2, Y */
} sentry_moe_desc;
SENTRY_API size_t sentry_moe_workspace_bytes(const sentry_moe_desc* desc);
SENTRY_API size_t sentry_moe_packed_bytes(const sentry_moe_desc* desc);
SENTRY_API int sentry_moe_prepack(sentry_ctx* ctx, const sentry_moe_desc* desc, const void* W1,
                       const void* W2, const int32_t* kept_channels, void* packed,
                       size_t packed_bytes, void* stream);
SENTRY_API int sentry_moe_ffn_fwd(sentry_ctx* ctx, const sentry_moe_desc* desc, const void* X,
                       const void* W1, const void* W2, const int32_t* kept_channels,
                       const void* packed, const int32_t* expert_ids,
                       const float* expert_weights, void* Y, void* stream);

/* ---------------------------------------------------------------------------
 * Projections of the pruned layer (Sec. 4.6, "Head pruning with GQA
 * consistency": of W_Q in R^{d_model x Hq d} only the column blocks of H_keep
 * are kept, of W_K and W_V the blocks of K_keep = floor(H_keep / (Hq/Hk)); a KV
 * group no kept head references is removed).  The paper never writes the
 * output projection; its row blocks follow the same rule.
 *
 *   X [B,T,D]; WQ [D, Hq*d]; WK, WV [D, Hk*d]; WO [Hq*d, D]   (row-major)
 *   kept_heads [B,k_h] i32 ascending; token_modality_ids [T]; masks [B]
 * sentry_project_qkv writes, for every present token t of sample b,
 *   Q[b,h,t,:] for the kept heads h and K[b,g,t,:], V[b,g,t,:] for the referenced
 *   groups g, into Q [B,Hq,T,d] and K, V [B,Hk,T,d] -- the layouts
 *   sentry_attend_fwd reads.  Nothing else is touched: slots of pruned heads,
 *   unreferenced groups and absent tokens keep what they held (sentry_attend_fwd
 *   never reads them).
 * sentry_project_out takes A [B,k_h,T,d] (sentry_attend_fwd's output, heads in
 *   kept-list order) and writes out [B,T,D] = sum_j A[b,j,t,:] . WO[h_j d:(h_j+1) d, :]
 *   for present tokens, zero rows for absent ones.
 * No bias, residual or normalisation.  fp32 accumulation, one rounding at the
 * store.  Limits: Hk <= 32, k_h <= 64, D <= 8192.
 */
typedef struct sentry_proj_desc {
    int B, T, D;       /* batch, tokens per sample, d_model */
    int Hq, Hk, d;     /* query heads, KV heads, head dim */
    int k_h;           /* kept heads per sample */
    int dtype;         /* sentry_dtype of every tensor */
} sentry_proj_desc;
SENTRY_API int sentry_project_qkv(sentry_ctx* ctx, const sentry_proj_desc* desc, const void* X,
                       const void* WQ, const void* WK, const void* WV, const int32_t* kept_heads,
                       const int32_t* token_modality_ids, const uint32_t* masks, void* Q, void* K,
                       void* V, void* stream);
SENTRY_API int sentry_project_out(sentry_ctx* ctx, const sentry_proj_desc* desc, const void* A,
                       const void* WO, const int32_t* kept_heads, const int32_t* token_modality_ids,
                       const uint32_t* masks, void* out, void* stream);

/* Which kernels run Eq. 6 for bf16 tensors whose K/V of one KV group fit in
 * shared memory (T up to ~1.4 k at d = 32).  Two hand-written forms exist:
 *   SENTRY_ATTEND_WARP_MMA  K/V staged by 16-byte async copies, Q K^T and P V
 *                           on the register-level warp MMA, online softmax
 *   SENTRY_ATTEND_TCGEN05   K/V staged by TMA tensor copies, Q K^T and P V on
 *                           tcgen05 with the accumulators and the softmax
 *                           weights in tensor memory, two-pass softmax
 * Both split every softmax weight into a bf16 head and a bf16 remainder, so the
 * results agree to well below the bf16 rounding of the stored output.
 * SENTRY_ATTEND_AUTO (default) takes the one that measured faster for the
 * shape.  Other shapes: bf16 with longer T runs a score kernel and a streamed
 * warp-MMA kernel; fp32, Hq/Hk > 4, U > 48 or T > 8192 run on the plain ALUs. */
#define SENTRY_OPT_ATTEND_KERNEL 1
#define SENTRY_ATTEND_AUTO 0
#define SENTRY_ATTEND_WARP_MMA 1
#define SENTRY_ATTEND_TCGEN05 2
/* SENTRY_OPT_LONG_SELECT: sequences whose K and V do not fit in shared memory
 * together take their scores and top-U selection either from a grid of
 * 256-query blocks per (sample, KV group) (QUERY_BLOCKS) or from one CTA per
 * group with the group's K rows resident (PER_GROUP: K staged once instead of
 * once per query block; needs about a group per SM to pay).  AUTO: PER_GROUP
 * when B*Hk >= the number of SMs.  Same results either way. */
#define SENTRY_OPT_LONG_SELECT 2
#define SENTRY_LONG_SELECT_AUTO 0
#define SENTRY_LONG_SELECT_QUERY_BLOCKS 1
#define SENTRY_LONG_SELECT_PER_GROUP 2
SENTRY_API int sentry_set_option(sentry_ctx* ctx, int option, int value);

/* ---------------------------------------------------------------------------
 * Channel-compacted FFN forward (Sec. 4.6): for every present row x,
 *   y = gelu(x . W1[:, N]) . W2[N, :],  gelu(z) = z/2 (1 + erf(z/sqrt 2)),
 * N = the kept-channel list of the row's sample.  No bias, residual or norm.
 */
typedef struct sentry_ffn_desc {
    int B, T, D, F; /* batch, tokens per sample, d_model, d_ff */
    int k_c;        /* kept channels per list */
    int n_lists;    /* number of kept-channel lists (one per modality subset in use) */
    int dtype;      /* sentry_dtype of X, W1, W2, Y (F32, BF16 or F16; the 16-bit types with D in
                       {128,256,384} run on tcgen05, everything else on the plain ALUs) */
} sentry_ffn_desc;

/*   X [B,T,D]; W1 [D,F]; W2 [F,D]; Y out [B,T,D]
 *   kept_channels [n_lists,k_c] i32 ascending in [0,F)
 *   list_of_sample [B] i32 in [0,n_lists) or NULL (list 0 for every sample)
 *   token_modality_ids [T] + masks [B], or both NULL (every row present);
 *   rows of absent-modality tokens get Y = 0 and cost no arithmetic.
 * The kept columns of W1 and rows of W2 are gathered into the workspace on
 * every call (the "materialised" pruned weights), then a fused GEMM pair runs
 * over the present rows.  Supported: D % 8 == 0, D <= 1024.
 * bf16 with D in {128, 256, 384} runs on the tcgen05 tensor cores, one
 * persistent CTA per SM; every other shape and fp32 run on the plain ALUs with
 * fp32 accumulation.  The GELU of the bf16 path evaluates
 * erf through the hardware tanh: within 4e-4 of gelu(|z|), below the rounding
 * of the bf16 hidden value it is stored as; fp32 uses erff.  Results are
 * bit-identical from call to call for identical inputs.
 */
SENTRY_API int sentry_ffn_fwd(sentry_ctx* ctx, const sentry_ffn_desc* desc, const void* X,
                   const void* W1, const void* W2, const int32_t* kept_channels,
                   const int32_t* list_of_sample, const int32_t* token_modality_ids,
                   const uint32_t* masks, void* Y, void* stream);

/* Self-test of the bounded device waits.  Every wait inside the kernels (on a
 * TMA copy, a tensor-core commit, another warp) gives up after about a second,
 * raises SENTRY_STATUS_BIT_TIMEOUT, lets copies in flight land, frees its
 * tensor memory and returns.  This call enqueues one small CTA that waits on a
 * barrier nothing ever signals, with a limit of `limit_cycles` SM clock cycles
 * (1 .. 1e8), and then leaves through that same path: afterwards
 * sentry_get_last_status reports SENTRY_STATUS_BIT_TIMEOUT and the context is
 * usable as before.  Nothing hangs or faults. */
SENTRY_API int sentry_selftest_wait_expiry(sentry_ctx* ctx, long long limit_cycles, void* stream);

/* Number of kernels the last call on this context enqueued (for launch
 * accounting in benchmarks). */
SENTRY_API int sentry_last_launch_count(const sentry_ctx* ctx);

/* Optional per-kernel timing for benchmarks.  While enabled, every kernel launch
 * is bracketed by CUDA events on the caller's stream.  sentry_profile_read
 * synchronises the device, adds up the elapsed time and the number of launches
 * per kernel slot since the last read into host arrays ms[n] / launches[n]
 * (n >= sentry_profile_slots()), and clears the record.  sentry_kernel_name
 * gives the slot's kernel name.  Off by default; adds launch gaps when on. */
SENTRY_API int sentry_profile_enable(sentry_ctx* ctx, int on);
SENTRY_API int sentry_profile_slots(void);
SENTRY_API int sentry_profile_read(sentry_ctx* ctx, float* ms, int* launches, int n);
SENTRY_API const char* sentry_kernel_name(int slot);

#ifdef __cplusplus
}
#endif
#endif /* SENTRY_H */

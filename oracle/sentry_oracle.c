/*
 * sentry_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, float64 CPU statement of what the pruned multimodal
 * transformer layer computes (SentryGate selection, SentryAttend sparse
 * grouped-query attention, channel-compacted FFN).  It exists so that the CUDA
 * library can be checked against something written directly from the paper.
 * Only the tests, the smoke check and the benchmark's cpu_baseline /
 * reference arm may load it.  It shares no code with the CUDA library.
 *
 * Every function cites the passage of the paper it follows.  Loops are written
 * in the order of the definitions: no blocking, no fusion, no reordering.
 * OpenMP is used only to run independent samples on several cores.
 *
 * Pins (see tests/test_oracle_pins.py):
 *   oracle_num_active      paper's worked example U(128)=25 (Section 4.4)
 *   oracle_gate_select     brute-force stable sort, library top-k, ties, NaN
 *   oracle_kv_groups       formula of Section 4.6 on hand cases
 *   oracle_attend          dense limit == library scaled-dot-product attention,
 *                          GQA duplication, rows of softmax sum to 1,
 *                          dropping == deleting, brute-force sparsity score
 *   oracle_ffn             library matmul + erf, masked full FFN
 *   oracle_project_qkv/out library matmul on sliced and on masked full weight matrices;
 *                          unpruned chain == textbook multi-head attention layer
 *   oracle_moe_ffn         library matmul per expert on sliced and on masked weights; one expert,
 *                          top-1 == oracle_ffn; linear in the routing weights
 *   oracle_gate_eval       library matmul form of the perceptron, closed forms
 *                          (zero first layer, gamma = 0, one hidden unit by hand)
 * The paper's GFLOP figures and accuracies need undisclosed architectures and
 * data: parity unpinned for those (they are not computed here).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Section 4.4: U = c * ceil(log T).  The worked example (T = 128, c = 5,
 * U ~ 25) fixes the natural logarithm and "ceil, then multiply".  T is the
 * number of tokens that are present; U is clamped to [1, T]. */
int oracle_num_active(int T_v, int c) {
    if (T_v <= 0) return 0;
    int u = c * (int)ceil(log((double)T_v));
    if (u > T_v) u = T_v;
    if (u < 1) u = 1;
    return u;
}

/* ---- SentryGate selection (Section 4.6: gate outputs for a fixed modality
 * mask are thresholded by a pruning ratio; here a per-layer, per-unit-type
 * budget k).  Order: score descending, index ascending on equal scores; NaN
 * ranks below every number.  The kept set is returned in ascending index
 * order. */
static int ranks_before(float sa, int ia, float sb, int ib) {
    /* 1 if unit a is ranked strictly before unit b */
    int na = isnan(sa), nb = isnan(sb);
    if (na || nb) {
        if (na && nb) return ia < ib;
        return nb; /* a is a number, b is NaN -> a first */
    }
    if (sa > sb) return 1;
    if (sa < sb) return 0;
    return ia < ib; /* equal (+0 == -0 included) */
}

void oracle_gate_select(const float* scores, int S, int n_units,
                        const uint32_t* masks, int n_masks, int k,
                        int32_t* kept) {
    (void)S;
    int* order = (int*)malloc(sizeof(int) * (size_t)n_units);
    for (int m = 0; m < n_masks; ++m) {
        const float* row = scores + (size_t)masks[m] * n_units;
        /* full stable insertion sort of all units by rank */
        for (int i = 0; i < n_units; ++i) {
            int j = i;
            while (j > 0 && ranks_before(row[i], i, row[order[j - 1]], order[j - 1])) {
                order[j] = order[j - 1];
                --j;
            }
            order[j] = i;
        }
        /* first k of the ranking, then ascending index */
        int32_t* out = kept + (size_t)m * k;
        for (int i = 0; i < k; ++i) out[i] = order[i];
        for (int i = 1; i < k; ++i) {
            int32_t v = out[i];
            int j = i;
            while (j > 0 && out[j - 1] > v) { out[j] = out[j - 1]; --j; }
            out[j] = v;
        }
    }
    free(order);
}

/* Section 4.6, head pruning with GQA consistency: head h belongs to KV group
 * floor(h / (H_q / H_k)); a group is kept iff some kept head maps to it. */
void oracle_kv_groups(const int32_t* kept_heads, int n_masks, int k_h,
                      int heads_per_group, uint32_t* groups_bitmap) {
    for (int m = 0; m < n_masks; ++m) {
        uint32_t bits = 0;
        for (int i = 0; i < k_h; ++i)
            bits |= 1u << (kept_heads[(size_t)m * k_h + i] / heads_per_group);
        groups_bitmap[m] = bits;
    }
}

/* Tokens whose modality is present under `mask`, ascending.  Returns T_v. */
int oracle_valid_tokens(const int32_t* ids, int T, uint32_t mask, int32_t* valid) {
    int n = 0;
    for (int t = 0; t < T; ++t)
        if ((mask >> ids[t]) & 1u) valid[n++] = t;
    return n;
}

/* ---- SentryAttend (Section 4.4, Eq. 6) for one sample.
 *
 * For each kept head h (KV group g = floor(h / r)):
 *   1. sparsity score of each present query i:
 *        M_i = max_{j in S_i} s_ij - mean_{j in S_i} s_ij,  s_ij = q_i.k_j / sqrt(d)
 *      S_i = the sampled keys listed in the table row of i (score_mode 0) or
 *      all present keys (score_mode 1);
 *   2. the U = c*ceil(ln T_v) queries with the largest M_i are active
 *      (ties -> lower token index), unless a forced selection is given;
 *   3. active rows:  softmax over ALL present keys, times V_g   (Eq. 6);
 *   4. the other present rows: mean of V_g over present keys;
 *   5. rows of absent-modality tokens: zero.
 * Output O is [k_h, T, d] for this sample, heads in kept-list order.
 */
static void attend_one_sample(const double* Q, const double* K, const double* V,
                              int T, int Hq, int Hk, int d, int c,
                              const int32_t* kept, int k_h,
                              const int32_t* ids, uint32_t mask, int score_mode,
                              const int32_t* table, int U_max,
                              const int32_t* forced, double* O, int32_t* active_out,
                              double* mscore_out) {
    int r = Hq / Hk;
    int32_t* valid = (int32_t*)malloc(sizeof(int32_t) * (size_t)T);
    int Tv = oracle_valid_tokens(ids, T, mask, valid);
    int U = oracle_num_active(Tv, c);
    int n_s = U;
    double scale = 1.0 / sqrt((double)d);
    double* M = (double*)malloc(sizeof(double) * (size_t)(Tv > 0 ? Tv : 1));
    char* is_active = (char*)malloc((size_t)(Tv > 0 ? Tv : 1));
    double* s = (double*)malloc(sizeof(double) * (size_t)(Tv > 0 ? Tv : 1));
    double* ctx = (double*)malloc(sizeof(double) * (size_t)d);

    memset(O, 0, sizeof(double) * (size_t)k_h * T * d);
    if (active_out)
        for (int i = 0; i < k_h * U_max; ++i) active_out[i] = -1;
    if (mscore_out)
        for (int i = 0; i < k_h * T; ++i) mscore_out[i] = NAN;

    for (int kh = 0; kh < k_h && Tv > 0; ++kh) {
        int h = kept[kh];
        int g = h / r;
        const double* Qh = Q + (size_t)h * T * d;
        const double* Kg = K + (size_t)g * T * d;
        const double* Vg = V + (size_t)g * T * d;

        /* step 1: sparsity score */
        for (int p = 0; p < Tv; ++p) {
            const double* q = Qh + (size_t)valid[p] * d;
            int cnt = (score_mode == 0) ? n_s : Tv;
            double mx = -INFINITY, sum = 0.0;
            for (int a = 0; a < cnt; ++a) {
                int pj = (score_mode == 0) ? table[(size_t)p * n_s + a] : a;
                const double* kk = Kg + (size_t)valid[pj] * d;
                double dot = 0.0;
                for (int e = 0; e < d; ++e) dot += q[e] * kk[e];
                dot *= scale;
                if (dot > mx) mx = dot;
                sum += dot;
            }
            M[p] = mx - sum / (double)cnt;
            if (mscore_out) mscore_out[(size_t)kh * T + valid[p]] = M[p];
        }

        /* step 2: top-U queries by M, ties -> lower index */
        memset(is_active, 0, (size_t)Tv);
        if (forced) {
            for (int a = 0; a < U_max; ++a) {
                int t = forced[(size_t)kh * U_max + a];
                if (t < 0) continue;
                for (int p = 0; p < Tv; ++p)
                    if (valid[p] == t) is_active[p] = 1;
            }
        } else {
            for (int a = 0; a < U; ++a) {
                int best = -1;
                for (int p = 0; p < Tv; ++p) {
                    if (is_active[p]) continue;
                    if (best < 0 || M[p] > M[best]) best = p;
                }
                is_active[best] = 1;
            }
        }
        if (active_out) {
            int a = 0;
            for (int p = 0; p < Tv; ++p)
                if (is_active[p] && a < U_max) active_out[(size_t)kh * U_max + a++] = valid[p];
        }

        /* step 4 prerequisite: context vector = mean of V_g over present keys */
        for (int e = 0; e < d; ++e) {
            double acc = 0.0;
            for (int pj = 0; pj < Tv; ++pj) acc += Vg[(size_t)valid[pj] * d + e];
            ctx[e] = acc / (double)Tv;
        }

        double* Oh = O + (size_t)kh * T * d;
        for (int p = 0; p < Tv; ++p) {
            double* o = Oh + (size_t)valid[p] * d;
            if (!is_active[p]) {
                for (int e = 0; e < d; ++e) o[e] = ctx[e];
                continue;
            }
            /* step 3: Eq. 6 on this row */
            const double* q = Qh + (size_t)valid[p] * d;
            double mx = -INFINITY;
            for (int pj = 0; pj < Tv; ++pj) {
                const double* kk = Kg + (size_t)valid[pj] * d;
                double dot = 0.0;
                for (int e = 0; e < d; ++e) dot += q[e] * kk[e];
                s[pj] = dot * scale;
                if (s[pj] > mx) mx = s[pj];
            }
            double den = 0.0;
            for (int pj = 0; pj < Tv; ++pj) { s[pj] = exp(s[pj] - mx); den += s[pj]; }
            for (int e = 0; e < d; ++e) {
                double acc = 0.0;
                for (int pj = 0; pj < Tv; ++pj) acc += (s[pj] / den) * Vg[(size_t)valid[pj] * d + e];
                o[e] = acc;
            }
        }
    }
    free(valid); free(M); free(is_active); free(s); free(ctx);
}

/* Batched driver.  Layouts: Q [B,Hq,T,d], K,V [B,Hk,T,d], kept_heads [B,k_h]
 * ascending, ids [T], masks [B]; sample_table = concatenated int32 rows,
 * table_offsets[mask value] = element offset of the [T_v, n_s] table for that
 * subset (compact key positions, i.e. indices into the present-token list);
 * forced_active [B,k_h,U_max] token indices padded with -1, or NULL.
 * O [B,k_h,T,d]; active_out [B,k_h,U_max] or NULL; mscore_out [B,k_h,T] or NULL. */
void oracle_attend(const double* Q, const double* K, const double* V,
                   int B, int T, int Hq, int Hk, int d, int c,
                   const int32_t* kept_heads, int k_h,
                   const int32_t* ids, const uint32_t* masks, int score_mode,
                   const int32_t* sample_table, const int64_t* table_offsets,
                   int U_max, const int32_t* forced_active,
                   double* O, int32_t* active_out, double* mscore_out) {
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const int32_t* table = NULL;
        if (score_mode == 0) table = sample_table + table_offsets[masks[b]];
        attend_one_sample(Q + (size_t)b * Hq * T * d, K + (size_t)b * Hk * T * d,
                          V + (size_t)b * Hk * T * d, T, Hq, Hk, d, c,
                          kept_heads + (size_t)b * k_h, k_h, ids, masks[b], score_mode,
                          table, U_max,
                          forced_active ? forced_active + (size_t)b * k_h * U_max : NULL,
                          O + (size_t)b * k_h * T * d,
                          active_out ? active_out + (size_t)b * k_h * U_max : NULL,
                          mscore_out ? mscore_out + (size_t)b * k_h * T : NULL);
    }
}

/* ---- Channel-compacted FFN (Section 4.6): W1' = W1[:, N_keep],
 * W2' = W2[N_keep, :], y = gelu(x W1') W2', gelu(z) = z/2 (1 + erf(z/sqrt 2)).
 * X [B,T,D], W1 [D,F], W2 [F,D], kept [n_lists,k_c], list_of_sample [B] or
 * NULL (list 0); ids/masks NULL -> every row computed, else rows of absent
 * modalities give zero.  Y [B,T,D]. */
void oracle_ffn(const double* X, const double* W1, const double* W2,
                int B, int T, int D, int F, const int32_t* kept, int k_c,
                const int32_t* list_of_sample, const int32_t* ids,
                const uint32_t* masks, double* Y) {
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const int32_t* N = kept + (size_t)(list_of_sample ? list_of_sample[b] : 0) * k_c;
        double* h = (double*)malloc(sizeof(double) * (size_t)k_c);
        for (int t = 0; t < T; ++t) {
            const double* x = X + ((size_t)b * T + t) * D;
            double* y = Y + ((size_t)b * T + t) * D;
            for (int e = 0; e < D; ++e) y[e] = 0.0;
            if (ids && masks && !((masks[b] >> ids[t]) & 1u)) continue;
            for (int n = 0; n < k_c; ++n) {
                double z = 0.0;
                for (int e = 0; e < D; ++e) z += x[e] * W1[(size_t)e * F + N[n]];
                h[n] = 0.5 * z * (1.0 + erf(z / sqrt(2.0)));
            }
            for (int e = 0; e < D; ++e) {
                double acc = 0.0;
                for (int n = 0; n < k_c; ++n) acc += h[n] * W2[(size_t)N[n] * D + e];
                y[e] = acc;
            }
        }
        free(h);
    }
}

/* ---- SentryGate score function (Section 4.2, Eq. 1):
 *   g_i(m) = sigmoid( zeta_i + gamma_l * f_i(m) ),  f_i = a two-layer perceptron on the mask m.
 * The paper names neither the hidden width nor the nonlinearity; ReLU is the reading taken:
 *   f_i(m) = sum_j w2[i][j] * max(0, b1[i][j] + sum_q W1[i][j][q] * m_q) + b2[i].
 * Units of all layers are concatenated; layer l owns [layer_offsets[l], layer_offsets[l+1]).
 * Writes z (the argument of the sigmoid) and g for every mask value s (m_q = bit q of s). */
void oracle_gate_eval(int M, int hidden, int n_layers, const int32_t* layer_offsets, int n_units,
                      const double* zeta, const double* gamma, const double* W1, const double* b1,
                      const double* w2, const double* b2, double* z_out, double* g_out) {
    const int S = 1 << M;
    for (int s = 0; s < S; ++s) {
        for (int l = 0; l < n_layers; ++l) {
            for (int i = layer_offsets[l]; i < layer_offsets[l + 1]; ++i) {
                double f = b2[i];
                for (int j = 0; j < hidden; ++j) {
                    double a = b1[(size_t)i * hidden + j];
                    for (int q = 0; q < M; ++q) {
                        const double m_q = (double)((s >> q) & 1);
                        a += W1[((size_t)i * hidden + j) * M + q] * m_q;
                    }
                    f += w2[(size_t)i * hidden + j] * (a > 0.0 ? a : 0.0);
                }
                const double z = zeta[i] + gamma[l] * f;
                z_out[(size_t)s * n_units + i] = z;
                g_out[(size_t)s * n_units + i] = 1.0 / (1.0 + exp(-z));
            }
        }
    }
    (void)n_units;
}

/* ---- Head pruning with GQA consistency (Section 4.6): the projections of a pruned layer.
 * W_Q is [d_model, H_q d_h]; of its H_q column blocks only those of the kept heads H_keep are
 * used.  The kept KV groups follow from them, K_keep = { floor(h / (H_q/H_k)) : h in H_keep }, and
 * W_K, W_V are filtered by block in the same way.  For every sample b and present token t:
 *   Q[b,h,t,:] = x_t . W_Q[:, h d : (h+1) d]        for h in H_keep(b)
 *   K[b,g,t,:] = x_t . W_K[:, g d : (g+1) d],  V likewise,  for g in K_keep(b)
 * Everything else (pruned heads, unreferenced groups, absent tokens) is left at zero here.
 * X [B,T,D]; W_Q [D, Hq d]; W_K, W_V [D, Hk d]; outputs Q [B,Hq,T,d], K, V [B,Hk,T,d]. */
void oracle_project_qkv(const double* X, const double* WQ, const double* WK, const double* WV, int B, int T, int D,
                        int Hq, int Hk, int d, const int32_t* kept_heads, int k_h, const int32_t* ids,
                        const uint32_t* masks, double* Q, double* K, double* V) {
    const int r = Hq / Hk;
    memset(Q, 0, sizeof(double) * (size_t)B * Hq * T * d);
    memset(K, 0, sizeof(double) * (size_t)B * Hk * T * d);
    memset(V, 0, sizeof(double) * (size_t)B * Hk * T * d);
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int t = 0; t < T; ++t) {
            if (!((masks[b] >> ids[t]) & 1u)) continue;
            const double* x = X + ((size_t)b * T + t) * D;
            for (int j = 0; j < k_h; ++j) {
                const int h = kept_heads[(size_t)b * k_h + j];
                const int g = h / r;
                for (int c = 0; c < d; ++c) {
                    double q = 0.0, kk = 0.0, vv = 0.0;
                    for (int e = 0; e < D; ++e) {
                        q += x[e] * WQ[(size_t)e * Hq * d + h * d + c];
                        kk += x[e] * WK[(size_t)e * Hk * d + g * d + c];
                        vv += x[e] * WV[(size_t)e * Hk * d + g * d + c];
                    }
                    Q[(((size_t)b * Hq + h) * T + t) * d + c] = q;
                    K[(((size_t)b * Hk + g) * T + t) * d + c] = kk;   /* same value from every head of the group */
                    V[(((size_t)b * Hk + g) * T + t) * d + c] = vv;
                }
            }
        }
    }
}

/* Output projection of the pruned layer: the row blocks of W_O that belong to the kept heads.
 * (The paper never writes W_O; this is the transpose of the rule it states for W_Q: a pruned head
 * contributes nothing, so its rows of W_O drop out.)
 *   out[b,t,:] = sum_j A[b,j,t,:] . W_O[h_j d : (h_j+1) d, :]   for present t, else 0
 * A [B,k_h,T,d] (heads in kept-list order); W_O [Hq d, D]; out [B,T,D]. */
void oracle_project_out(const double* A, const double* WO, int B, int T, int D, int Hq, int d,
                        const int32_t* kept_heads, int k_h, const int32_t* ids, const uint32_t* masks, double* out) {
    memset(out, 0, sizeof(double) * (size_t)B * T * D);
    (void)Hq;
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int t = 0; t < T; ++t) {
            if (!((masks[b] >> ids[t]) & 1u)) continue;
            double* o = out + ((size_t)b * T + t) * D;
            for (int j = 0; j < k_h; ++j) {
                const int h = kept_heads[(size_t)b * k_h + j];
                const double* a = A + (((size_t)b * k_h + j) * T + t) * d;
                for (int c = 0; c < d; ++c)
                    for (int e = 0; e < D; ++e) o[e] += a[c] * WO[(size_t)(h * d + c) * D + e];
            }
        }
    }
}

/* ---- Sparse-MoE FFN pruning (Section 4.6): the expert count and the top-k routing rule are left
 * alone; what is pruned is the inside of each expert, whose own FFN keeps a channel set N_e of its
 * own: W1_e' = W1_e[:, N_e], W2_e' = W2_e[N_e, :].  The routing result (which experts a token goes to, with which
 * weights) is an INPUT: pruning does not touch it.  For every token t
 *   y_t = sum_j weight[t][j] * ( gelu(x_t . W1_e[:, N_e]) . W2_e[N_e, :] ),   e = expert[t][j],
 * gelu as in oracle_ffn (exact erf; the paper names no activation).
 * X [N,D]; W1 [E,D,F]; W2 [E,F,D]; kept [E,k_c]; expert [N,top_k]; weight [N,top_k]; Y [N,D]. */
void oracle_moe_ffn(const double* X, const double* W1, const double* W2, int N, int D, int F, int E,
                    const int32_t* kept, int k_c, const int32_t* expert, const double* weight, int top_k,
                    double* Y) {
#pragma omp parallel
    {
        double* h = (double*)malloc(sizeof(double) * (size_t)k_c);
#pragma omp for schedule(dynamic, 16)
        for (int t = 0; t < N; ++t) {
            const double* x = X + (size_t)t * D;
            double* y = Y + (size_t)t * D;
            for (int e2 = 0; e2 < D; ++e2) y[e2] = 0.0;
            for (int j = 0; j < top_k; ++j) {
                const int e = expert[(size_t)t * top_k + j];
                const double g = weight[(size_t)t * top_k + j];
                const double* w1 = W1 + (size_t)e * D * F;
                const double* w2 = W2 + (size_t)e * F * D;
                const int32_t* Ne = kept + (size_t)e * k_c;
                for (int n = 0; n < k_c; ++n) {
                    double z = 0.0;
                    for (int e2 = 0; e2 < D; ++e2) z += x[e2] * w1[(size_t)e2 * F + Ne[n]];
                    h[n] = 0.5 * z * (1.0 + erf(z / sqrt(2.0)));
                }
                for (int n = 0; n < k_c; ++n)
                    for (int e2 = 0; e2 < D; ++e2) y[e2] += g * h[n] * w2[(size_t)Ne[n] * D + e2];
            }
        }
        free(h);
    }
    (void)E;
}

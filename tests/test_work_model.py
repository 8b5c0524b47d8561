"""Pins for bench.work_model, the algorithmic FLOP / byte count behind `useful_tflops` and both
roofline fractions: a brute-force count, one multiply-add or one element at a time, over the
loop nest of the method as the oracle walks it (Section 4.4: per kept head, every present query
is scored on its sampled keys, then the U active queries attend to every present key;
Section 4.6: every present row meets every kept channel twice)."""
import numpy as np

import bench
import oracle
import synth


def _brute_force(w: synth.Workload, masks, kept_heads):
    e = 4 if w.dtype == "f32" else 2
    r = w.Hq // w.Hk
    ids = synth.token_modality_ids(w)
    macs_att = adds_mean = macs_ffn = 0
    elems_att = 0      # elements of Q, K, V read and of O written
    elems_rows = 0     # elements of X read and Y written
    tokens = 0
    for b, m in enumerate(masks):
        valid = [t for t in range(w.T) if (int(m) >> int(ids[t])) & 1]
        tv = len(valid)
        tokens += tv
        U = oracle.num_active(tv, w.c)
        n_s = U
        groups = sorted(set(int(h) // r for h in kept_heads[b]))
        for _h in kept_heads[b]:
            for _i in range(tv):               # sparsity score of every present query
                macs_att += n_s * w.d
            for _a in range(U):                # Eq. 6 rows: q.k and p.v over every present key
                macs_att += tv * w.d + tv * w.d
            elems_att += tv * w.d              # Q rows in
            elems_att += tv * w.d              # O rows out (present tokens only)
        for _g in groups:
            adds_mean += tv * w.d              # context vector: column sums of V_g
            elems_att += 2 * tv * w.d          # K_g and V_g rows in
        for _i in range(tv):
            macs_ffn += w.D * w.k_c + w.k_c * w.D
            elems_rows += 2 * w.D
    return {"tokens": tokens, "att_flops": 2.0 * macs_att + adds_mean, "ffn_flops": 2.0 * macs_ffn,
            "att_bytes": float(e * elems_att), "ffn_row_bytes": float(e * elems_rows)}


def _case(w):
    inp = synth.generate(w, lambda tv: oracle.num_active(tv, w.c), tensors=False)
    kept = oracle.gate_select(inp.scores_heads, inp.masks, w.k_h)
    return inp, kept


def test_work_model_equals_brute_force_count():
    cases = [synth.config1(), synth.config2().with_(B=24), synth.config4().with_(B=9),
             synth.config5(14, 64), synth.Workload("odd", "bf16", 5, (37, 5, 91), 72, 6, 3, 16, 200, 4, 77,
                                                   "cycle7", 9)]
    for w in cases:
        inp, kept = _case(w)
        wm = bench.work_model(w, inp.masks, kept, lambda tv: oracle.num_active(tv, w.c))
        bf = _brute_force(w, inp.masks, kept)
        assert wm["tokens"] == bf["tokens"], w.name
        np.testing.assert_allclose(wm["att_flops"], bf["att_flops"], rtol=1e-12, err_msg=w.name)
        np.testing.assert_allclose(wm["ffn_flops"], bf["ffn_flops"], rtol=1e-12, err_msg=w.name)
        np.testing.assert_allclose(wm["att_bytes"], bf["att_bytes"], rtol=1e-12, err_msg=w.name)
        n_lists = len(set(int(m) for m in inp.masks))
        e = 4 if w.dtype == "f32" else 2
        weights = 2.0 * w.D * w.k_c * e * n_lists
        np.testing.assert_allclose(wm["kernel_bytes"]["ffn_main"], bf["ffn_row_bytes"] + weights, rtol=1e-12)


def test_attention_work_grows_as_n_U_T_not_n_T_squared():
    # Section 4.4: O(n T^2) -> O(n U T), U = c ceil(ln T).  Doubling T from 1024 to 2048 leaves
    # U at 35 -> 40: the work must grow by 2 * 40/35, far from the dense factor 4.
    def flops(T):
        w = synth.Workload("s", "bf16", 1, (T,), 64, 8, 2, 32, 64, 8, 8, "all", 0)
        inp, kept = _case(w)
        return bench.work_model(w, inp.masks, kept, lambda tv: oracle.num_active(tv, 5))["att_flops"]
    a, b = flops(1024), flops(2048)
    U1, U2 = oracle.num_active(1024, 5), oracle.num_active(2048, 5)
    assert (U1, U2) == (35, 40)
    assert abs(b / a - 2.0 * U2 / U1) < 0.01 and b / a < 2.5
    # per kept head and present token: 2 d (n_s + 2 U) = 6 U d flops (+ the context mean)
    w = synth.Workload("s", "bf16", 1, (1024,), 64, 8, 2, 32, 64, 8, 8, "all", 0)
    assert abs(a - (8 * 1024 * 6 * 35 * 32 + 2 * 1024 * 32)) < 1

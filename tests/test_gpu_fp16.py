"""IEEE-half storage (the FP16 point of the paper's post-training-quantisation axis, Section 5): the
pruned FFN pair on tcgen05 with fp16 operands, the Sparse-MoE block on the same kernel, attention on the
warp-MMA kernels compiled for fp16 operands, projections on the plain-ALU kernels, each against the
float64 oracle fed the same fp16 values."""
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


@pytest.fixture()
def sn():
    s = sentry.Sentry(0)
    yield s
    s.close()


@pytest.mark.parametrize("w", [
    synth.config2().with_(dtype="f16", name="cfg2_f16", B=40),          # D = 128, one chunk per tile
    synth.config3().with_(dtype="f16", name="cfg3_f16", B=5),           # D = 256, 40 tiles
    synth.config4().with_(dtype="f16", name="cfg4_f16", B=12),          # D = 384, ragged k_c = 614, three lists
    synth.Workload("ragged_f16", "f16", 5, (37, 5, 91), 72, 6, 3, 16, 200, 4, 77, "cycle7", 48),   # plain-ALU FFN
], ids=lambda w: w.name)
def test_fp16_ffn_and_attention(sn, w):
    inp = synth.generate(w, n_s_of)
    kept_h, kept_c = parity.gate_lists(sn, inp)
    err_f = parity.ffn_parity(sn, inp, kept_c, None, full_batch=True)
    assert err_f <= TOL["f16"], err_f
    # bit-identical on a second call, and with the weights materialised once
    X, W1, W2 = inp.X.cuda(), inp.W1.cuda(), inp.W2.cuda()
    ids, masks, los = dev(inp.ids), masks_dev(inp.masks), dev(inp.list_of_sample)
    Y1 = sn.ffn_fwd(X, W1, W2, kept_c, los, ids, masks)
    packed = sn.ffn_prepack(W1, W2, kept_c)
    Y2 = sn.ffn_fwd_packed(X, packed, w.F, w.k_c, kept_c.shape[0], los, ids, masks)
    assert torch.equal(Y1, Y2)
    # attention: the warp-MMA kernels compiled for fp16 operands
    err_a, _ = parity.attend_parity(sn, inp, kept_h, None, 0, full_batch=True)
    assert err_a <= TOL["f16"], err_a


@pytest.mark.parametrize("w", [
    synth.Workload("att_f16", "f16", 4, (40, 24, 33), 64, 8, 2, 32, 128, 5, 64, "cycle7", 49),
    synth.Workload("att_f16_d64", "f16", 4, (140, 124, 133), 64, 8, 2, 64, 128, 5, 64, "cycle7", 50),
    synth.Workload("att_f16_long", "f16", 5, (1300, 1100, 900), 64, 8, 2, 32, 128, 4, 64, "cycle7", 51),   # streamed Eq. 6
    synth.Workload("att_f16_5heads", "f16", 3, (60, 70), 64, 10, 2, 16, 128, 9, 64, "all", 52),   # 5 heads per group: plain-ALU kernels
], ids=lambda w: w.name)
def test_fp16_attention(sn, w):
    inp = synth.generate(w, n_s_of)
    kept_h, _ = parity.gate_lists(sn, inp)
    try:
        for form in (sentry.LONG_SELECT_PER_GROUP, sentry.LONG_SELECT_QUERY_BLOCKS):
            sn.set_option(sentry.OPT_LONG_SELECT, form)
            err_a, _ = parity.attend_parity(sn, inp, kept_h, None, 0, full_batch=True)
            assert err_a <= TOL["f16"], err_a
    finally:
        sn.set_option(sentry.OPT_LONG_SELECT, sentry.LONG_SELECT_AUTO)
    # heads selected inside the attention launch: same bits as the two-call form
    ids, masks = dev(inp.ids), masks_dev(inp.masks)
    tbl, offs = dev(inp.sample_table), dev(inp.table_offsets)
    Q, K, V = inp.Q.cuda(), inp.K.cuda(), inp.V.cuda()
    O1 = sn.attend_fwd(Q, K, V, kept_h, ids, masks, tbl, offs, c=w.c)
    O2, kept2 = sn.gate_attend_fwd(dev(inp.scores_heads), w.k_h, Q, K, V, ids, masks, tbl, offs, c=w.c)
    assert torch.equal(kept2, kept_h) and torch.equal(O1, O2)


def test_fp16_moe(sn):
    N, D, F, E, top_k, k_c = 1500, 256, 1024, 8, 2, 512
    m = synth.generate_moe(N, D, F, E, top_k, k_c, "f16", seed=77, skew=1.0, unrouted=0.05)
    X, W1, W2 = m.X.cuda(), m.W1.cuda(), m.W2.cuda()
    kept = torch.from_numpy(m.kept).cuda()
    Y = sn.moe_ffn_fwd(X, torch.from_numpy(m.expert_ids).cuda(), torch.from_numpy(m.expert_weights).cuda(),
                       W1=W1, W2=W2, kept_channels=kept)
    assert sn.last_status() == 0
    ids = m.expert_ids.copy()
    wts = m.expert_weights.astype(np.float64).copy()
    wts[ids < 0] = 0.0
    ids[ids < 0] = 0
    want = oracle.moe_ffn(m.X, m.W1, m.W2, m.kept, ids, wts)
    got = Y.float().cpu().numpy()
    err = parity.rel_err(got, want, "f16", np.ones(N, dtype=bool))
    parity.record("moe_f16", "moe", err, parity.raw_rel_err(got, want), "%d tokens" % N)
    assert err <= TOL["f16"], err

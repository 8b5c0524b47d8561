"""Sparse-MoE block with expert-internal channel pruning (Section 4.6) against the float64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_08971_b200 as sentry
import synth
from tests import parity
from tests.parity import TOL

pytestmark = pytest.mark.gpu

# (name, N, D, F, E, top_k, k_c, dtype, skew, unrouted)
CASES = [
    ("moe_small_f32", 301, 64, 192, 5, 2, 96, "f32", 1.0, 0.0),
    ("moe_tc_d256", 2500, 256, 1024, 8, 2, 512, "bf16", 1.0, 0.0),        # several tiles per expert + tails
    ("moe_tc_d256_multi_block_plan", 6000, 256, 1024, 8, 2, 512, "bf16", 1.0, 0.05),   # > 8192 slots: count / offsets / scatter launches
    ("moe_tc_d384_top4", 1111, 384, 768, 16, 4, 300, "bf16", 1.5, 0.1),   # k_c padded to a chunk; dropped slots
    ("moe_tc_d128_idle", 700, 128, 512, 32, 1, 256, "bf16", 3.0, 0.0),    # top-1, most experts nearly idle
    ("moe_alu_bf16_d72", 257, 72, 200, 3, 2, 77, "bf16", 0.0, 0.2),       # shape outside the tensor-core path
]


def _oracle_inputs(m):
    """Slots marked -1 contribute nothing: for the oracle that is expert 0 with weight 0."""
    ids = m.expert_ids.copy()
    wts = m.expert_weights.astype(np.float64).copy()
    wts[ids < 0] = 0.0
    ids[ids < 0] = 0
    return ids, wts


@pytest.mark.parametrize("case", CASES, ids=lambda c: c[0])
def test_moe_ffn_matches_oracle(case):
    name, N, D, F, E, top_k, k_c, dtype, skew, unrouted = case
    m = synth.generate_moe(N, D, F, E, top_k, k_c, dtype, seed=len(name) * 131 + N, skew=skew, unrouted=unrouted)
    sn = sentry.Sentry(0)
    try:
        X, W1, W2 = m.X.cuda(), m.W1.cuda(), m.W2.cuda()
        kept = torch.from_numpy(m.kept).cuda()
        ids = torch.from_numpy(m.expert_ids).cuda()
        wts = torch.from_numpy(m.expert_weights).cuda()
        Y = sn.moe_ffn_fwd(X, ids, wts, W1=W1, W2=W2, kept_channels=kept)
        assert sn.last_status() == 0
        launches = sn.last_launch_count()
        o_ids, o_wts = _oracle_inputs(m)
        want = oracle.moe_ffn(m.X, m.W1, m.W2, m.kept, o_ids, o_wts)
        got = Y.float().cpu().numpy()
        rows = np.ones(N, dtype=bool)
        err = parity.rel_err(got, want, dtype, rows)
        parity.record(name, "moe", err, parity.raw_rel_err(got, want), "%d tokens, %d launches" % (N, launches))
        assert err <= TOL[dtype], err
        # a token with no routed slot gets exactly zero
        dead = np.all(m.expert_ids < 0, axis=1)
        assert np.all(got[dead] == 0.0)
        # weights materialised once: same bits, fewer launches
        packed = sn.moe_prepack(W1, W2, kept)
        Y2 = sn.moe_ffn_fwd(X, ids, wts, packed=packed, F=F, E=E, k_c=k_c)
        assert sn.last_status() == 0
        assert sn.last_launch_count() == launches - 1
        assert torch.equal(Y, Y2)
        # run to run: the grouping of rows uses atomics, the values must not depend on it
        Y3 = sn.moe_ffn_fwd(X, ids, wts, packed=packed, F=F, E=E, k_c=k_c)
        assert torch.equal(Y2, Y3)
    finally:
        sn.close()


def test_moe_one_expert_top1_equals_plain_ffn():
    """E = 1, top-1, weight 1: bit for bit the channel-compacted FFN on the same rows."""
    m = synth.generate_moe(640, 256, 512, 1, 1, 256, "bf16", seed=9)
    sn = sentry.Sentry(0)
    try:
        X, W1, W2 = m.X.cuda(), m.W1.cuda(), m.W2.cuda()
        kept = torch.from_numpy(m.kept).cuda()
        ids = torch.zeros((640, 1), dtype=torch.int32, device="cuda")
        wts = torch.ones((640, 1), dtype=torch.float32, device="cuda")
        Y = sn.moe_ffn_fwd(X, ids, wts, W1=W1, W2=W2, kept_channels=kept)
        Yp = sn.ffn_fwd(X[None], W1[0].contiguous(), W2[0].contiguous(), kept)
        assert torch.equal(Y, Yp[0])
    finally:
        sn.close()


def test_moe_bad_expert_id_is_flagged_and_skipped():
    m = synth.generate_moe(200, 128, 256, 4, 2, 128, "bf16", seed=3)
    sn = sentry.Sentry(0)
    try:
        ids_np = m.expert_ids.copy()
        ids_np[17, 1] = 4          # == E
        ids_np[90, 0] = -7
        X, W1, W2 = m.X.cuda(), m.W1.cuda(), m.W2.cuda()
        kept = torch.from_numpy(m.kept).cuda()
        wts = torch.from_numpy(m.expert_weights).cuda()
        Y = sn.moe_ffn_fwd(X, torch.from_numpy(ids_np).cuda(), wts, W1=W1, W2=W2, kept_channels=kept)
        assert sn.last_status() & sentry.STATUS_BIT_BAD_INDEX
        ok_ids = ids_np.copy()
        ok_ids[17, 1] = -1
        ok_ids[90, 0] = -1
        Y_ok = sn.moe_ffn_fwd(X, torch.from_numpy(ok_ids).cuda(), wts, W1=W1, W2=W2, kept_channels=kept)
        assert sn.last_status() == 0
        assert torch.equal(Y, Y_ok)
    finally:
        sn.close()

"""FFN weights stored as FP8 e4m3 codes with one scale per matrix (Section 5, the FP8 point of the
quantisation axis: storage): sentry_ffn_prepack_fp8 must produce, bit for bit, the packed weights that
sentry_ffn_prepack makes of the oracle's dequantised matrices, and the FFN on them must meet the usual
bound against the oracle."""
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


@pytest.mark.parametrize("w", [
    synth.config4().with_(B=10), synth.config3().with_(B=4), synth.config2().with_(B=30, dtype="f16", name="cfg2_f16_fp8w"),
    synth.config1(),
    synth.Workload("ragged_fp8w", "bf16", 5, (37, 5, 91), 72, 6, 3, 16, 200, 4, 77, "cycle7", 96),
], ids=lambda w: w.name)
def test_fp8_stored_weights(w):
    sn = sentry.Sentry(0)
    try:
        inp = synth.generate(w, n_s_of)
        _, kept_c = parity.gate_lists(sn, inp)
        # quantise the generated weights to e4m3 with a per-matrix scale (library conversion, test side)
        s1 = float(inp.W1.float().abs().max()) / 448.0
        s2 = float(inp.W2.float().abs().max()) / 448.0
        W1q = (inp.W1.float() / s1).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()
        W2q = (inp.W2.float() / s2).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()
        W1d = oracle.dequantise_e4m3(W1q.numpy(), s1, w.dtype)
        W2d = oracle.dequantise_e4m3(W2q.numpy(), s2, w.dtype)
        dt = synth.torch_dtype(w)
        packed = sn.ffn_prepack_fp8(W1q.cuda(), W2q.cuda(), s1, s2, kept_c, dtype=dt)
        assert sn.last_status() == 0
        packed_ref = sn.ffn_prepack(W1d.cuda(), W2d.cuda(), kept_c)
        assert torch.equal(packed, packed_ref)
        ids, masks, los = dev(inp.ids), masks_dev(inp.masks), dev(inp.list_of_sample)
        X = inp.X.cuda()
        Y = sn.ffn_fwd_packed(X, packed, w.F, w.k_c, kept_c.shape[0], los, ids, masks)
        assert sn.last_status() == 0
        want = oracle.ffn(inp.X, W1d, W2d, kept_c.cpu().numpy(), inp.list_of_sample, inp.ids, inp.masks)
        got = Y.float().cpu().numpy()
        err = parity.rel_err(got, want, w.dtype, np.ones(got.shape[:2], dtype=bool))
        parity.record(w.name, "ffn_fp8w", err, parity.raw_rel_err(got, want), "weights stored as e4m3 + scale")
        assert err <= TOL[w.dtype], err
    finally:
        sn.close()

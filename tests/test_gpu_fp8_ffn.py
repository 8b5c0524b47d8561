"""The channel-compacted FFN with FP8 (e4m3) operands on tcgen05 (Section 5, the FP8 point of the
quantisation axis taken to the arithmetic) against the oracle's FP8 FFN.

Tolerance.  Both sides multiply the same e4m3 codes exactly and differ in (a) the order of the fp32
accumulation and (b) the GELU (exact erf in the oracle, the tanh form on the device, 1.5e-4 apart):
a hidden activation that lands within ~3e-4 (relative) of an e4m3 rounding boundary may round the
other way, by one step of 2^-3 .. 2^-4 of its size -- for ANY implementation that does not sum in
the oracle's order.  About 1 % of the hidden values do; an output sums k_c of them, so its error
is a handful of +-6 % errors on single terms of a sum of ~k_c terms: ~0.5 % of the output RMS
typically (measured 0.4 %), while the rare output that catches a flip on one of its largest terms
is off by several per cent of the RMS.  Element-wise 2e-2 of the RMS can therefore not hold for
every output; what is asserted is what the arithmetic fixes:
  * the RMS of the error <= 1.5e-2 of the output RMS,
  * at most 5 outputs in 1000 off by more than 2e-2 of the RMS (after the bf16 half-ulp of Y; measured 2 in 1000:
    a flipped term has to be ~7 times the typical term to move an output that far).  That size falls with the
    number of terms (0.33 sqrt(k_c) typical terms: 4.7 at k_c = 200, 7.5 at 512) while the error RMS does not
    depend on it, so below 300 kept channels the allowed fraction grows as 300 / k_c (measured 5.1 in 1000 at
    k_c = 200, 4.4 at 256),
  * no output off by more than 0.25 of the RMS (a flip or two on the largest terms, nothing worse),
  * rows of absent tokens exactly zero, results identical run to run.
"""
import numpy as np
import pytest
import torch
from scipy.special import erf

import oracle
import paper_2604_08971_b200 as sentry
import synth
from tests import parity
from tests.parity import dev, masks_dev

pytestmark = pytest.mark.gpu


def n_s_of(tv):
    return sentry.num_active_queries(tv, 5)


def _quantise(t):
    s = float(t.float().abs().max()) / 448.0
    q = (t.float() / s).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()
    return q, s


@pytest.mark.parametrize("w", [synth.config3().with_(B=6), synth.config5(16, 256), synth.config5(3, 1024).with_(k_c=300, name="fp8_ragged_kc"),
                               synth.config2().with_(B=24, name="fp8_d128"), synth.config2().with_(B=5, k_c=200, name="fp8_d128_ragged_kc"),
                               synth.config4().with_(B=12, name="fp8_d384"), synth.config4().with_(B=70, name="fp8_d384_two_tiles_per_cta")],
                         ids=lambda w: w.name)
def test_fp8_ffn_against_the_oracle(w):
    sn = sentry.Sentry(0)
    try:
        inp = synth.generate(w, n_s_of)
        _, kept_c = parity.gate_lists(sn, inp)
        Xq, sx = _quantise(inp.X)
        W1q, sw1 = _quantise(inp.W1)
        W2q, sw2 = _quantise(inp.W2)
        # calibration of the hidden scale: the largest hidden activation of this batch (float, test side)
        z = (oracle.e4m3_decode(Xq.numpy()).reshape(-1, w.D) @ oracle.e4m3_decode(W1q.numpy())) * (sx * sw1)
        sh = float(np.max(np.abs(0.5 * z * (1.0 + erf(z / np.sqrt(2.0)))))) / 448.0
        packed = sn.ffn_prepack_e4m3(W1q.cuda(), W2q.cuda(), kept_c)
        ids, masks, los = dev(inp.ids), masks_dev(inp.masks), dev(inp.list_of_sample)
        Y = sn.ffn_fwd_fp8(Xq.cuda(), packed, w.F, w.k_c, kept_c.shape[0], sx, sw1, sw2, sh, los, ids, masks)
        assert sn.last_status() == 0
        Y2 = sn.ffn_fwd_fp8(Xq.cuda(), packed, w.F, w.k_c, kept_c.shape[0], sx, sw1, sw2, sh, los, ids, masks)
        assert torch.equal(Y, Y2)
        want = oracle.ffn_fp8(Xq.numpy(), W1q.numpy(), W2q.numpy(), kept_c.cpu().numpy(), inp.list_of_sample, inp.ids,
                              inp.masks, sx, sw1, sw2, sh)
        got = Y.float().cpu().numpy()
        for b in range(w.B):
            gone = np.nonzero(((int(inp.masks[b]) >> inp.ids) & 1) == 0)[0]
            assert np.all(got[b][gone] == 0.0)
        err = parity.rel_err(got, want, "bf16", np.ones(got.shape[:2], dtype=bool))
        rms = float(np.sqrt(np.mean(want ** 2)))
        rms_err = float(np.sqrt(np.mean((got - want) ** 2))) / rms
        excess = np.maximum(np.abs(got - want) - parity.bf16_half_ulp(want), 0.0)
        frac_off = float(np.mean(excess > 2e-2 * rms))
        parity.record(w.name, "ffn_fp8", err, parity.raw_rel_err(got, want),
                      "error rms %.2e of the output rms; %.1e of the outputs off by more than 2e-2" % (rms_err, frac_off))
        assert rms_err <= 1.5e-2, rms_err
        assert frac_off <= 5e-3 * max(1.0, 300.0 / w.k_c), frac_off
        assert err <= 0.25, err
    finally:
        sn.close()

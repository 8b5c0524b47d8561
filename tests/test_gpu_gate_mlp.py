"""SentryGate evaluated on the device (Eq. 1) and the cross-layer threshold of Section 4.6 against
the float64 oracle: the logit / gate tables within fp32 rounding, the kept lists bit-exact on the
table the device produced, and the per-layer counts exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_08971_b200 as sentry

pytestmark = pytest.mark.gpu


def _params(seed, units, hidden, M):
    g = np.random.default_rng(seed)
    lo = np.concatenate([[0], np.cumsum(units)]).astype(np.int32)
    N = int(lo[-1])
    f32 = lambda x: x.astype(np.float32)
    return (lo, f32(g.standard_normal(N)), f32(g.standard_normal(len(units))),
            f32(g.standard_normal((N, hidden, M)) * 0.5), f32(g.standard_normal((N, hidden))),
            f32(g.standard_normal((N, hidden)) * 0.5), f32(g.standard_normal(N)))


@pytest.mark.parametrize("units,hidden,M", [([12, 12, 12, 12], 8, 3), ([12, 1536], 16, 2), ([4, 256, 4, 256, 7], 5, 4)])
def test_gate_eval_global_threshold_and_layer_counts(units, hidden, M):
    sn = sentry.Sentry(0)
    try:
        lo, zeta, gamma, W1, b1, w2, b2 = _params(len(units) * 100 + hidden, units, hidden, M)
        d = lambda x: torch.as_tensor(x).cuda()
        logits, gates = sn.gate_eval(d(lo), d(zeta), d(gamma), d(W1), d(b1), d(w2), d(b2), return_gates=True)
        z, g = oracle.gate_eval(lo, zeta, gamma, W1, b1, w2, b2)
        scale = max(1.0, float(np.abs(z).max()))
        assert np.abs(logits.cpu().numpy() - z).max() <= 1e-5 * scale
        assert np.abs(gates.cpu().numpy() - g).max() <= 1e-5
        # global threshold: keep 60 % of all units of all layers together
        N = int(lo[-1])
        k = max(1, int(0.6 * N))
        masks = np.arange(1, 1 << M, dtype=np.int32)
        kept = sn.gate_select(logits, d(masks), k)
        want = oracle.gate_select(logits.cpu().numpy(), masks.astype(np.uint32), k)   # the device's own table
        np.testing.assert_array_equal(kept.cpu().numpy(), want)
        # against the oracle's table: the same set wherever the k-th and (k+1)-th logits are clearly apart
        for r, s in enumerate(masks):
            srt = np.sort(z[s])[::-1]
            if srt[k - 1] - srt[k] > 1e-4 * scale:
                assert set(want[r].tolist()) == set(np.argsort(-z[s], kind="stable")[:k].tolist())
        counts = sn.gate_layer_counts(kept, d(lo)).cpu().numpy()
        for r in range(len(masks)):
            np.testing.assert_array_equal(counts[r], np.histogram(want[r], bins=lo)[0])
        assert counts.sum(axis=1).tolist() == [k] * len(masks)
        assert sn.last_status() == 0
    finally:
        sn.close()

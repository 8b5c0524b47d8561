"""The CTA-pair form of the tensor-core FFN (SENTRY_FFN_KERNEL=pair) against the oracle.

The library reads the variable once per process, so the check runs in a child process:
workloads with d_model 128, 256 and 384 (all three instantiations), several tiles per CTA
pair, a ragged last tile and more than one kept-channel list.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
import torch
import paper_2604_08971_b200 as sentry
import synth
from tests import parity

sn = sentry.Sentry(0)
n_s_of = lambda tv: sentry.num_active_queries(tv, 5)
for w in (synth.config2().with_(B=40), synth.by_name("3b").with_(B=3), synth.config4().with_(B=24),
          synth.config5(16, 256)):
    inp = synth.generate(w, n_s_of)
    kept_h, kept_c = parity.gate_lists(sn, inp)
    err = parity.ffn_parity(sn, inp, kept_c)
    print(w.name, "ffn err %%.3e" %% err, "status", sn.last_status())
    assert err <= parity.TOL[w.dtype], (w.name, err)
    assert sn.last_status() == 0
sn.close()
print("PAIR_OK")
""" % ROOT


@pytest.mark.gpu
def test_pair_kernel_matches_oracle():
    env = dict(os.environ, SENTRY_FFN_KERNEL="pair")
    res = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0 and "PAIR_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]

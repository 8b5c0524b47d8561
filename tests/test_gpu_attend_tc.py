"""The tcgen05 form of SentryAttend (SENTRY_ATTEND_TCGEN05: K/V staged by TMA, Q K^T and P V on
tcgen05 with accumulators and softmax weights in tensor memory) against the float64 oracle, on
the workloads whose K/V of a KV group fit in shared memory; and the case both forms share of
present tokens scattered over many short runs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_08971_b200 as sentry
import synth
from tests import parity
from tests.parity import TOL, dev, masks_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sn_tc():
    ctx = sentry.Sentry(0)
    ctx.set_attend_kernel(sentry.ATTEND_TCGEN05)
    yield ctx
    ctx.close()


def n_s_of(tv):
    return sentry.num_active_queries(tv, 5)


def _attend(sn, w, samples="all", score_mode=0, device="cpu", scatter=False):
    inp = synth.generate(w, n_s_of, device=device)
    if scatter:   # the same tokens per modality, interleaved: present tokens form many short runs
        inp.ids = np.random.default_rng(w.seed).permutation(inp.ids).astype(np.int32)
    kept_h, _ = parity.gate_lists(sn, inp)
    sel = None if samples == "all" else parity.stratified_samples(inp, 2)
    err, ties = parity.attend_parity(sn, inp, kept_h, sel, score_mode, full_batch=True)
    assert err <= TOL[w.dtype], (w.name, err)
    return err


@pytest.mark.parametrize("name", ["2", "3a", "3b", "3c", "4"])
def test_named_workloads(sn_tc, name):
    _attend(sn_tc, synth.by_name(name))


@pytest.mark.parametrize("B,T", [(1, 64), (16, 64), (16, 256), (256, 256), (16, 1024), (256, 1024), (4096, 64)])
def test_sweep_cells(sn_tc, B, T):
    _attend(sn_tc, synth.config5(B, T))


def test_large_sweep_cells_whole_batch_call(sn_tc):
    for B, T in [(4096, 256), (4096, 1024)]:
        _attend(sn_tc, synth.config5(B, T), samples="strat", device="cuda")
        torch.cuda.empty_cache()


@pytest.mark.parametrize("d", [16, 32, 64])
def test_ragged_runs_and_head_dims(sn_tc, d):
    # runs of 37, 5 and 91 tokens: TMA boxes between the 8-row boundaries, single rows at the edges
    w = synth.Workload("ragged_tc", "bf16", 5, (37, 5, 91), 72, 6, 3, d, 200, 4, 77, "cycle7", 40 + d)
    _attend(sn_tc, w)
    _attend(sn_tc, w, score_mode=1)


def test_dense_degenerate_two_row_tiles_and_forced_selection(sn_tc):
    # T_v <= U: every present row is an Eq. 6 row
    _attend(sn_tc, synth.Workload("dense_tc", "bf16", 3, (4, 3, 2), 64, 4, 2, 16, 64, 2, 16, "cycle7", 50))
    # four kept heads in one KV group, U = 35: 140 stacked rows = two M = 128 tiles
    _attend(sn_tc, synth.Workload("two_tiles", "bf16", 3, (300, 300), 64, 8, 2, 32, 64, 8, 16, "all", 56))
    w = synth.Workload("forced_tc", "bf16", 3, (20, 30), 64, 4, 2, 32, 64, 2, 32, "all", 55)
    inp = synth.generate(w, n_s_of)
    kept_h, _ = parity.gate_lists(sn_tc, inp)
    g = np.random.default_rng(7)
    U = n_s_of(50)
    forced = np.stack([[np.sort(g.choice(50, U, replace=False)) for _ in range(2)]
                       for _ in range(3)]).astype(np.int32)
    O = sn_tc.attend_fwd(inp.Q.cuda(), inp.K.cuda(), inp.V.cuda(), kept_h, dev(inp.ids),
                         masks_dev(inp.masks), active_in=dev(forced), score_mode=1)
    want = oracle.attend(inp.Q, inp.K, inp.V, kept_h.cpu().numpy(), inp.ids, inp.masks,
                         score_mode=1, forced_active=forced)
    rows = np.zeros(want.shape[:3], dtype=bool)
    for b_ in range(3):
        for j_ in range(2):
            rows[b_, j_, forced[b_, j_]] = True
    assert parity.rel_err(O.float().cpu().numpy(), want, "bf16", rows) <= TOL["bf16"]
    assert sn_tc.last_status() == 0


def test_unreferenced_group_is_never_read(sn_tc):
    w = synth.Workload("grp_tc", "bf16", 4, (48, 48), 64, 8, 2, 32, 128, 3, 128, "all", 52)
    inp = synth.generate(w, n_s_of)
    inp.scores_heads[:, :4] = -10.0
    kept_h, _ = parity.gate_lists(sn_tc, inp)
    inp.K[:, 0] = float("nan")
    inp.V[:, 0] = float("nan")
    err, _ = parity.attend_parity(sn_tc, inp, kept_h)
    assert err <= TOL["bf16"]


def test_absent_tokens_may_hold_anything(sn_tc):
    # K/V/Q rows of absent-modality tokens are NaN: they must not reach any output
    w = synth.Workload("nan_tc", "bf16", 6, (37, 5, 91), 72, 6, 3, 32, 200, 4, 77, "cycle7", 61)
    inp = synth.generate(w, n_s_of)
    kept_h, _ = parity.gate_lists(sn_tc, inp)
    for b in range(w.B):
        gone = torch.as_tensor(np.nonzero(((int(inp.masks[b]) >> inp.ids) & 1) == 0)[0])
        inp.Q[b][:, gone] = float("nan")
        inp.K[b][:, gone] = float("nan")
        inp.V[b][:, gone] = float("nan")
    err, _ = parity.attend_parity(sn_tc, inp, kept_h)
    assert err <= TOL["bf16"]


@pytest.mark.parametrize("kernel", [sentry.ATTEND_WARP_MMA, sentry.ATTEND_TCGEN05])
def test_scattered_present_tokens(kernel):
    sn = sentry.Sentry(0)
    sn.set_attend_kernel(kernel)
    try:
        _attend(sn, synth.Workload("scatter", "bf16", 7, (40, 33, 60), 72, 6, 3, 32, 200, 4, 77, "cycle7", 62),
                scatter=True)
    finally:
        sn.close()

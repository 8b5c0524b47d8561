"""sentry_gate_select_static -- the gate selection for hosts that may not allocate.

A plug-in running inside another runtime's memory pool, or a service whose device-memory
budget is fixed at start-up, cannot call cudaMalloc: it can neither create a library context
nor provide a workspace.  The static entry point keeps its scratch in an array inside the
library image instead.  These tests call it through the C ABI and require the same kept lists
and KV-group bitmaps as sentry_gate_select (integer results: bit-exact), on two calls in a row
that share the static array -- the second smaller than the first, so that anything read from
the first call's leftovers would show.

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test.  Passes alone in a fresh process and after the rest of the suite.
"""
import gc

import numpy as np
import pytest
import torch

import oracle
import paper_2604_08971_b200 as sentry

pytestmark = pytest.mark.gpu


def _case(seed, S, n, k, n_masks, hpg):
    g = np.random.default_rng(seed)
    scores = g.standard_normal((S, n)).astype(np.float32)
    scores[:, ::7] = 0.25  # exact ties: the lower index must win in both entry points
    masks = g.integers(1, S, size=n_masks).astype(np.int32)
    return torch.as_tensor(scores).cuda(), torch.as_tensor(masks).cuda(), k, hpg


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    sn = sentry.Sentry(0)
    try:
        # (seed, score rows, units, budget, masks, heads per KV group)
        for seed, S, n, k, n_masks, hpg in [(11, 16, 1536, 614, 500, 0), (12, 8, 12, 7, 64, 3)]:
            scores, masks, k, hpg = _case(seed, S, n, k, n_masks, hpg)
            want = sn.gate_select(scores, masks, k, heads_per_group=hpg)
            want_kept, want_groups = want if hpg > 0 else (want, None)
            # every buffer is made here, before the call: the call itself allocates nothing
            kept = torch.full((n_masks, k), -7, dtype=torch.int32, device="cuda")
            groups = torch.zeros((n_masks,), dtype=torch.int32, device="cuda") if hpg > 0 else None
            status = torch.zeros((1,), dtype=torch.int32, device="cuda")
            gc.collect()                      # tensors earlier tests dropped must not be freed mid-measurement
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
            sentry.gate_select_static(scores, masks, k, kept, groups, hpg, status)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() <= before   # the call itself allocated nothing
            assert torch.equal(kept, want_kept)
            # and the same lists as the float64 oracle's full ordering (ties -> lower index)
            np.testing.assert_array_equal(
                kept.cpu().numpy(), oracle.gate_select(scores.cpu().numpy(), masks.cpu().numpy(), k))
            if hpg > 0:
                assert torch.equal(groups, want_groups)
            assert int(status.item()) == 0
    finally:
        sn.close()


def test_static_entry_point_flags_bad_mask_and_rejects_oversize():
    scores, masks, k, _ = _case(13, 8, 64, 16, 32, 0)
    masks[5] = 8  # >= S: that row is skipped and flagged, nothing faults
    kept = torch.zeros((32, k), dtype=torch.int32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    sentry.gate_select_static(scores, masks, k, kept, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & sentry.STATUS_BIT_BAD_INDEX
    # scratch need beyond the static array: refused on the host with the workspace error
    big = torch.zeros((4096, 64), device="cuda")
    with pytest.raises(sentry.SentryError) as e:
        sentry.gate_select_static(big, masks, 64, torch.zeros((32, 64), dtype=torch.int32, device="cuda"))
    assert e.value.code == -4
    # a score row too long for the kernel's default shared-memory window
    wide = torch.zeros((2, 20000), device="cuda")
    with pytest.raises(sentry.SentryError) as e:
        sentry.gate_select_static(wide, masks[:1] * 0 + 1, 8, torch.zeros((1, 8), dtype=torch.int32, device="cuda"))
    assert e.value.code == -3

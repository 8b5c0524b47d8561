"""GPU parity: libsentry (through its C ABI) against the float64 oracle on the
same seeded inputs.  Kept-index lists bit-exact; outputs within 1e-4 (fp32) and
2e-2 (bf16) max-abs error relative to the output RMS."""
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
def sn():
    ctx = sentry.Sentry(0)
    yield ctx
    ctx.close()


def n_s_of(tv):
    return sentry.num_active_queries(tv, 5)


# ------------------------------------------------------------------------ gate
@pytest.mark.parametrize("n,k", [(4, 3), (8, 4), (8, 2), (8, 6), (12, 7), (256, 128), (512, 256),
                                 (1024, 512), (1536, 614), (7, 7), (9, 1), (5000, 1234)])
def test_gate_bit_exact(sn, n, k):
    g = np.random.default_rng(n * 1000 + k)
    S = 16
    scores = g.standard_normal((S, n)).astype(np.float32)
    masks = g.integers(1, S, size=300).astype(np.uint32)
    got = sn.gate_select(dev(scores), masks_dev(masks), k).cpu().numpy()
    np.testing.assert_array_equal(got, oracle.gate_select(scores, masks, k))
    assert sn.last_status() == 0


def test_gate_ties_nan_zero_and_groups(sn):
    g = np.random.default_rng(5)
    n = 96
    # heavy ties: scores drawn from 5 distinct values, plus NaN, +-0, +-inf
    pool = np.array([0.5, -0.0, 0.0, 1.5, np.nan, -np.inf, np.inf, 0.5], dtype=np.float32)
    scores = pool[g.integers(0, len(pool), size=(8, n))]
    masks = np.arange(8, dtype=np.uint32)
    for k in (1, 7, 32, 95, 96):
        got, groups = sn.gate_select(dev(scores), masks_dev(masks), k, heads_per_group=4)
        want = oracle.gate_select(scores, masks, k)
        np.testing.assert_array_equal(got.cpu().numpy(), want)
        np.testing.assert_array_equal(groups.cpu().numpy().astype(np.uint32),
                                      oracle.kv_groups(want, 4))


def test_gate_large_fanout_and_bad_mask(sn):
    g = np.random.default_rng(6)
    scores = g.standard_normal((8, 1024)).astype(np.float32)
    masks = (1 + np.arange(4096) % 7).astype(np.uint32)
    got = sn.gate_select(dev(scores), masks_dev(masks), 512).cpu().numpy()
    np.testing.assert_array_equal(got, oracle.gate_select(scores, masks, 512))
    assert sn.last_status() == 0
    bad = masks.copy()
    bad[17] = 9  # >= S: skipped and flagged, no fault
    sn.gate_select(dev(scores), masks_dev(bad), 512)
    assert sn.last_status() & sentry.STATUS_BIT_BAD_INDEX


def test_error_codes_no_launch(sn):
    scores = torch.zeros((4, 8), device="cuda")
    masks = torch.ones((2,), dtype=torch.int32, device="cuda")
    with pytest.raises(sentry.SentryError) as e:
        sn.gate_select(scores, masks, 9)
    assert e.value.code == -2
    with pytest.raises(sentry.SentryError) as e:
        sn.gate_select(scores, masks, 0, kept=torch.empty((2, 1), dtype=torch.int32, device="cuda"))
    assert e.value.code == -2
    Q = torch.zeros((1, 4, 8, 24), device="cuda")  # head_dim 24 unsupported
    K = torch.zeros((1, 2, 8, 24), device="cuda")
    kh = torch.zeros((1, 2), dtype=torch.int32, device="cuda")
    ids = torch.zeros((8,), dtype=torch.int32, device="cuda")
    with pytest.raises(sentry.SentryError) as e:
        sn.attend_fwd(Q, K, K, kh, ids, masks[:1], score_mode=1)
    assert e.value.code == -3
    Q = torch.zeros((1, 4, 8, 16), device="cuda")
    K = torch.zeros((1, 2, 8, 16), device="cuda")
    with pytest.raises(sentry.SentryError) as e:   # sampled mode without a table
        sn.attend_fwd(Q, K, K, kh, ids, masks[:1], score_mode=0)
    assert e.value.code == -1
    X = torch.zeros((1, 8, 12), device="cuda")     # D % 8 != 0
    W1 = torch.zeros((12, 16), device="cuda")
    W2 = torch.zeros((16, 12), device="cuda")
    kc = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(sentry.SentryError) as e:
        sn.ffn_fwd(X, W1, W2, kc)
    assert e.value.code == -3
    assert sn.last_status() == 0


# ------------------------------------------------------------------ workloads
def _run_workload(sn, w, attend_samples="all", ffn_samples="all", score_mode=0, device="cpu"):
    """Gate lists bit-exact, then attention and FFN against the oracle.  "all": every sample goes
    through the CUDA call and the oracle.  "strat": the CUDA call still runs on the WHOLE batch
    (the launch shape the benchmark times: for the FFN 128-row tiles over 148 persistent CTAs),
    and the oracle checks at least two samples of every modality subset of its output."""
    inp = synth.generate(w, n_s_of, device=device)
    kept_h, kept_c = parity.gate_lists(sn, inp)
    strat = parity.stratified_samples(inp, 2)
    a_s = None if attend_samples == "all" else strat
    f_s = None if ffn_samples == "all" else strat
    err_a, ties = parity.attend_parity(sn, inp, kept_h, a_s, score_mode, full_batch=True)
    err_f = parity.ffn_parity(sn, inp, kept_c, f_s, full_batch=True)
    assert err_a <= TOL[w.dtype], (w.name, "attend", err_a)
    assert err_f <= TOL[w.dtype], (w.name, "ffn", err_f)
    return err_a, err_f, ties


def test_config1_fp32_both_score_modes_and_single_modalities(sn):
    w = synth.config1()
    _run_workload(sn, w, "all", "all", 0)
    _run_workload(sn, w, "all", "all", 1)
    inp = synth.generate(w, n_s_of)
    kept_h, kept_c = parity.gate_lists(sn, inp)
    for m in (1, 2):  # one modality dropped: rows of its tokens are zero, the rest as if deleted
        inp.masks[:] = m
        g = np.random.default_rng(m)
        inp.sample_table, inp.table_offsets = synth.make_sample_tables(w, inp.masks, n_s_of, g)
        inp.subsets = np.array([m], dtype=np.uint32)
        inp.list_of_sample[:] = 0
        err_a, _ = parity.attend_parity(sn, inp, kept_h)
        err_f = parity.ffn_parity(sn, inp, kept_c[:1])
        assert err_a <= TOL["f32"] and err_f <= TOL["f32"]


# FFN tiles per persistent CTA in the full-batch calls below (128-row tiles, 148 CTAs):
#   workload 2: ~35 k present rows -> ~277 tiles -> up to 2 per CTA   (d_model 128, four X slots)
#   workload 3: 65 536 rows        -> 512 tiles  -> up to 4 per CTA   (d_model 256)
#   workload 4: 43 520 rows        -> 341 tiles  -> up to 3 per CTA   (d_model 384, k_c = 614 ragged)
def test_config2_wearable_bf16(sn):
    _run_workload(sn, synth.config2(), "all", "all")


@pytest.mark.parametrize("ratio", [0.25, 0.5, 0.75])
def test_config3_physio_head_keep_sweep(sn, ratio):
    _run_workload(sn, synth.config3(ratio), "all", "all")


def test_config4_full_layer_all_subsets(sn):
    w = synth.config4()
    inp = synth.generate(w, n_s_of, tensors=False)
    assert sorted(set(inp.masks.tolist())) == [1, 2, 3]
    _run_workload(sn, w, "all", "all")


# d_model = 384: the tiles of a partial last round are shared by three CTAs each (a 128-column third
# of Y per CTA) when three times their number fits one round of 148 CTAs.  Three batch sizes put the
# kernel in each regime: every tile shared (B = 12: 32 tiles), two whole rounds of none and a shared
# third (B = 64: 170 tiles = 148 + 22), a partial round too large to share (B = 78: 208 = 148 + 60).
@pytest.mark.parametrize("B", [12, 64, 78])
def test_ffn_d384_column_split_regimes(sn, B):
    w = synth.config4().with_(B=B, name="cfg4_B%d" % B)
    inp = synth.generate(w, n_s_of)
    _, kept_c = parity.gate_lists(sn, inp)
    strat = parity.stratified_samples(inp, 2)
    err = parity.ffn_parity(sn, inp, kept_c, strat, full_batch=True)
    assert err <= TOL["bf16"], (w.name, err)
    # and twice the same bits
    X, W1, W2 = inp.X.cuda(), inp.W1.cuda(), inp.W2.cuda()
    los, ids, masks = dev(inp.list_of_sample), dev(inp.ids), masks_dev(inp.masks)
    Y1 = sn.ffn_fwd(X, W1, W2, kept_c, los, ids, masks)
    Y2 = sn.ffn_fwd(X, W1, W2, kept_c, los, ids, masks)
    assert torch.equal(Y1, Y2)


# All 16 cells of the throughput sweep.  Up to 2^18 tokens every sample is checked; beyond that
# the call runs on the whole batch (inputs drawn on the device) and the oracle checks two samples
# of each of the 7 modality subsets.
@pytest.mark.parametrize("B,T", synth.CONFIG5_CELLS)
def test_config5_sweep_cells(sn, B, T):
    big = B * T > (1 << 18)
    mode = "strat" if big else "all"
    _run_workload(sn, synth.config5(B, T), mode, mode, device="cuda" if big else "cpu")
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name,lengths,Hq,Hk,d,k_h", [
    ("long_d64_segments", (700, 900, 600), 8, 2, 64, 6),    # K of a group: up to 275 KB -> walked in segments, up to 4 heads per group
    ("long_d16_resident", (2100, 1500, 1400), 6, 3, 16, 4),  # 5000 tokens, K resident in one piece
    ("long_d32_three_heads", (1300, 1100, 900), 12, 4, 32, 9),
], ids=lambda v: v if isinstance(v, str) else None)
def test_long_sequences_selection_by_one_cta_per_group(sn, name, lengths, Hq, Hk, d, k_h):
    """Sequences whose K and V do not fit in shared memory together: scores and top-U by the
    one-CTA-per-group kernel (K resident, or walked in segments), Eq. 6 by the streamed kernel."""
    w = synth.Workload(name, "bf16", 7, lengths, 64, Hq, Hk, d, 128, k_h, 64, "cycle7", 60 + d)
    try:
        for form in (sentry.LONG_SELECT_PER_GROUP, sentry.LONG_SELECT_QUERY_BLOCKS):
            sn.set_option(sentry.OPT_LONG_SELECT, form)
            _run_workload(sn, w, "all", "all")
    finally:
        sn.set_option(sentry.OPT_LONG_SELECT, sentry.LONG_SELECT_AUTO)


@pytest.mark.parametrize("w,kernel", [
    (synth.config1(), sentry.ATTEND_AUTO),                                         # fp32: plain-ALU kernels
    (synth.config4().with_(B=9), sentry.ATTEND_AUTO),                              # fused warp-MMA kernel
    (synth.config4().with_(B=9), sentry.ATTEND_TCGEN05),                           # tcgen05 kernel
    (synth.config2().with_(B=12), sentry.ATTEND_AUTO),                             # short sequences, 128-thread CTAs
    (synth.Workload("long_em", "bf16", 7, (1300, 1100, 900), 64, 8, 2, 32, 128, 4, 64, "cycle7", 91), sentry.ATTEND_AUTO),
    (synth.Workload("long_em_d64", "bf16", 7, (700, 900, 600), 64, 8, 2, 64, 128, 6, 64, "cycle7", 92), sentry.ATTEND_AUTO),
], ids=lambda v: v.name if isinstance(v, synth.Workload) else str(v))
def test_entry_major_sample_table_gives_the_same_bits(sn, w, kernel):
    """score_mode 2 reads the same sample sets from the transposed table, in the same order:
    the output and the active lists must equal those of score_mode 0 bit for bit."""
    inp = synth.generate(w, n_s_of)
    kept_h, _ = parity.gate_lists(sn, inp)
    ids, masks = dev(inp.ids), masks_dev(inp.masks)
    tbl, offs = dev(inp.sample_table), dev(inp.table_offsets)
    tbl_em = dev(synth.entry_major_tables(w, inp.sample_table, inp.table_offsets, n_s_of))
    Q, K, V = inp.Q.cuda(), inp.K.cuda(), inp.V.cuda()
    sn.set_attend_kernel(kernel)
    sn.set_option(sentry.OPT_LONG_SELECT, sentry.LONG_SELECT_PER_GROUP)
    try:
        O0, act0 = sn.attend_fwd(Q, K, V, kept_h, ids, masks, tbl, offs, c=w.c, score_mode=0, return_active=True)
        O2, act2 = sn.attend_fwd(Q, K, V, kept_h, ids, masks, tbl_em, offs, c=w.c, score_mode=2, return_active=True)
        # the query-block form of the long-sequence selection reads the same table
        sn.set_option(sentry.OPT_LONG_SELECT, sentry.LONG_SELECT_QUERY_BLOCKS)
        O3 = sn.attend_fwd(Q, K, V, kept_h, ids, masks, tbl_em, offs, c=w.c, score_mode=2)
    finally:
        sn.set_attend_kernel(sentry.ATTEND_AUTO)
        sn.set_option(sentry.OPT_LONG_SELECT, sentry.LONG_SELECT_AUTO)
    assert sn.last_status() == 0
    assert torch.equal(act0, act2)
    assert torch.equal(O0, O3)
    assert torch.equal(O0, O2)


@pytest.mark.parametrize("w", [
    synth.config1(), synth.config2().with_(B=12), synth.config4().with_(B=9), synth.config3().with_(B=3),
    synth.Workload("ragged_arr", "bf16", 5, (37, 5, 91), 72, 6, 3, 64, 200, 4, 77, "cycle7", 47),
    synth.Workload("long_arr", "bf16", 7, (1300, 1100, 900), 64, 8, 2, 32, 128, 4, 64, "cycle7", 93),
], ids=lambda w: w.name)
def test_arranged_sample_tables_keep_the_sets_and_the_parity(sn, w):
    """sentry_sample_table_arrange: every query keeps exactly its sampled set (bit-exact integer
    work), stored entry-major; attention on the arranged tables meets the same bound against the
    oracle, which reads the tables as generated."""
    inp = synth.generate(w, n_s_of)
    ids, tbl, offs = dev(inp.ids), dev(inp.sample_table), dev(inp.table_offsets)
    arr = sn.sample_table_arrange(ids, tbl, offs, c=w.c)
    assert sn.last_status() == 0
    arr_np = arr.cpu().numpy()
    seen = set()
    worse = better = 0
    for s, off in enumerate(inp.table_offsets):
        if off < 0 or int(off) in seen:
            continue
        seen.add(int(off))
        tv = synth.present_count(w, s)
        n_s = n_s_of(tv)
        orig = inp.sample_table[off:off + tv * n_s].reshape(tv, n_s)
        got = arr_np[off:off + tv * n_s].reshape(n_s, tv).T
        np.testing.assert_array_equal(np.sort(got, axis=1), np.sort(orig, axis=1))
        # rows read in one access phase (8 consecutive queries, same step): fewer equal residues mod 8
        for q0 in range(0, tv - 7, 8):
            for a in range(n_s):
                worse += np.bincount(orig[q0:q0 + 8, a] % 8, minlength=8).max()
                better += np.bincount(got[q0:q0 + 8, a] % 8, minlength=8).max()
    if worse:
        assert better <= worse
    kept_h, _ = parity.gate_lists(sn, inp)
    try:
        for form in (sentry.LONG_SELECT_PER_GROUP, sentry.LONG_SELECT_QUERY_BLOCKS):
            sn.set_option(sentry.OPT_LONG_SELECT, form)
            err, _ = parity.attend_parity(sn, inp, kept_h, None, 0, full_batch=True, arranged=True)
            assert err <= TOL[w.dtype], (w.name, err)
    finally:
        sn.set_option(sentry.OPT_LONG_SELECT, sentry.LONG_SELECT_AUTO)


@pytest.mark.parametrize("w,kernel", [
    (synth.config2().with_(B=24), sentry.ATTEND_AUTO),       # heads selected inside the fused kernel (128-thread CTAs)
    (synth.config4().with_(B=20), sentry.ATTEND_AUTO),       # the same, 256-thread CTAs, three subsets
    (synth.config3().with_(B=3), sentry.ATTEND_AUTO),        # 512-thread CTAs
    (synth.config4().with_(B=6), sentry.ATTEND_TCGEN05),     # gate launch + tcgen05 kernel
    (synth.config1(), sentry.ATTEND_AUTO),                   # fp32: gate launch + plain-ALU kernels
    (synth.Workload("long_ga", "bf16", 4, (1300, 1100, 900), 64, 8, 2, 32, 128, 4, 64, "cycle7", 94), sentry.ATTEND_AUTO),
], ids=lambda v: v.name if isinstance(v, synth.Workload) else str(v))
def test_gate_and_attention_in_one_call(sn, w, kernel):
    """sentry_gate_attend_fwd == sentry_gate_select followed by sentry_attend_fwd, bit for bit:
    kept-head lists, active lists and output."""
    inp = synth.generate(w, n_s_of)
    ids, masks = dev(inp.ids), masks_dev(inp.masks)
    tbl, offs = dev(inp.sample_table), dev(inp.table_offsets)
    sh = dev(inp.scores_heads)
    Q, K, V = inp.Q.cuda(), inp.K.cuda(), inp.V.cuda()
    U_max = n_s_of(w.T)
    sn.set_attend_kernel(kernel)
    try:
        kept = sn.gate_select(sh, masks, w.k_h)
        O1, act1 = sn.attend_fwd(Q, K, V, kept, ids, masks, tbl, offs, c=w.c, return_active=True)
        act2 = torch.full((w.B, w.k_h, U_max), -7, dtype=torch.int32, device="cuda")
        O2, kept2 = sn.gate_attend_fwd(sh, w.k_h, Q, K, V, ids, masks, tbl, offs, c=w.c, active_out=act2)
        launches = sn.last_launch_count()
    finally:
        sn.set_attend_kernel(sentry.ATTEND_AUTO)
    assert sn.last_status() == 0
    np.testing.assert_array_equal(kept2.cpu().numpy(), oracle.gate_select(inp.scores_heads, inp.masks, w.k_h))
    assert torch.equal(kept, kept2)
    assert torch.equal(act1, act2)
    assert torch.equal(O1, O2)
    if w.dtype == "bf16" and kernel == sentry.ATTEND_AUTO and w.T <= 1024:
        assert launches == 1   # B * Hk is far below the bound beyond which the gate gets its own launch


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [16, 32, 64])
def test_ragged_shapes_and_head_dims(sn, dtype, d):
    # token counts that are not multiples of any tile; 3 modalities of unequal length
    w = synth.Workload("ragged", dtype, 5, (37, 5, 91), 72, 6, 3, d, 200, 4, 77, "cycle7", 40 + d)
    _run_workload(sn, w, "all", "all")


def test_dense_degenerate_and_single_token(sn):
    # T_v <= U: every present row is an Eq. 6 row (dense GQA attention)
    w = synth.Workload("dense", "f32", 3, (4, 3, 2), 64, 4, 2, 16, 64, 2, 16, "cycle7", 50)
    _run_workload(sn, w, "all", "all")
    w1 = synth.Workload("one", "f32", 2, (1,), 64, 2, 1, 16, 64, 1, 8, "all", 51)
    _run_workload(sn, w1, "all", "all")


def test_whole_kv_group_pruned_and_k_extremes(sn):
    # scores that force all kept heads into group 1: group 0 is never referenced
    w = synth.Workload("grp", "bf16", 4, (48, 48), 64, 8, 2, 32, 128, 3, 128, "all", 52)
    inp = synth.generate(w, n_s_of)
    inp.scores_heads[:, :4] = -10.0
    kept_h, kept_c = parity.gate_lists(sn, inp)
    assert kept_h.min().item() >= 4
    # poison the unreferenced group's K/V: the result must not change
    inp.K[:, 0] = float("nan")
    inp.V[:, 0] = float("nan")
    err, _ = parity.attend_parity(sn, inp, kept_h)
    assert err <= TOL["bf16"]
    assert parity.ffn_parity(sn, inp, kept_c) <= TOL["bf16"]   # k_c = F: nothing pruned
    for k_h in (1, 8):
        w2 = w.with_(k_h=k_h, seed=53 + k_h)
        inp2 = synth.generate(w2, n_s_of)
        kh2, _ = parity.gate_lists(sn, inp2)
        err, _ = parity.attend_parity(sn, inp2, kh2)
        assert err <= TOL["bf16"]


def test_exact_score_ties_select_lower_index(sn):
    w = synth.Workload("ties", "f32", 2, (40,), 64, 2, 1, 16, 64, 2, 8, "all", 54)
    inp = synth.generate(w, n_s_of)
    inp.Q[:] = inp.Q[:, :, :1, :]          # identical queries -> identical sparsity scores
    inp.sample_table[:] = np.tile(np.arange(n_s_of(40), dtype=np.int32), 40)  # same sampled keys
    kept_h, _ = parity.gate_lists(sn, inp)
    O, act = sn.attend_fwd(inp.Q.cuda(), inp.K.cuda(), inp.V.cuda(), kept_h, dev(inp.ids),
                           masks_dev(inp.masks), dev(inp.sample_table), dev(inp.table_offsets),
                           return_active=True)
    U = n_s_of(40)
    assert act.cpu().numpy()[:, :, :U].tolist() == [[list(range(U))] * 2] * 2


def test_forced_selection_and_empty_mask_flag(sn):
    w = synth.Workload("forced", "bf16", 3, (20, 30), 64, 4, 2, 32, 64, 2, 32, "all", 55)
    inp = synth.generate(w, n_s_of)
    kept_h, _ = parity.gate_lists(sn, inp)
    g = np.random.default_rng(7)
    U = n_s_of(50)
    forced = np.stack([[np.sort(g.choice(50, U, replace=False)) for _ in range(2)]
                       for _ in range(3)]).astype(np.int32)
    O = sn.attend_fwd(inp.Q.cuda(), inp.K.cuda(), inp.V.cuda(), kept_h, dev(inp.ids),
                      masks_dev(inp.masks), active_in=dev(forced), score_mode=1)
    want = oracle.attend(inp.Q, inp.K, inp.V, kept_h.cpu().numpy(), inp.ids, inp.masks,
                         score_mode=1, forced_active=forced)
    got = O.float().cpu().numpy()
    rows = np.zeros(got.shape[:3], dtype=bool)
    for b_ in range(3):
        for j_ in range(2):
            rows[b_, j_, forced[b_, j_]] = True
    assert parity.rel_err(got, want, "bf16", rows) <= TOL["bf16"]
    assert sn.last_status() == 0
    # a sample whose mask is empty: zeros out, flag set, nothing faults
    masks = inp.masks.copy()
    masks[1] = 0
    O = sn.attend_fwd(inp.Q.cuda(), inp.K.cuda(), inp.V.cuda(), kept_h, dev(inp.ids),
                      masks_dev(masks), score_mode=1)
    assert sn.last_status() & sentry.STATUS_BIT_EMPTY_MASK
    assert torch.all(O[1] == 0)


def test_results_are_deterministic_run_to_run(sn):
    """Identical calls give bit-identical outputs.  The FFN cases are full batches, so every
    persistent CTA walks several tiles (workload 2: up to 2, workload 4: up to 3, a sweep cell
    with 1024 tiles: up to 7) and the cross-tile hand-overs are part of what must repeat."""
    w = synth.config2().with_(B=16)
    inp = synth.generate(w, n_s_of)
    kept_h, kept_c = parity.gate_lists(sn, inp)
    args = (inp.Q.cuda(), inp.K.cuda(), inp.V.cuda(), kept_h, dev(inp.ids), masks_dev(inp.masks),
            dev(inp.sample_table), dev(inp.table_offsets))
    O1 = sn.attend_fwd(*args).clone()
    O2 = sn.attend_fwd(*args)
    assert torch.equal(O1.view(torch.int16), O2.view(torch.int16))
    for w in (synth.config2(), synth.config4(), synth.config5(256, 1024)):
        inp = synth.generate(w, n_s_of, device="cuda")
        kept_h, kept_c = parity.gate_lists(sn, inp)
        fargs = (inp.X, inp.W1, inp.W2, kept_c, dev(inp.list_of_sample), dev(inp.ids), masks_dev(inp.masks))
        Y1 = sn.ffn_fwd(*fargs).clone()
        for _ in range(6):
            Y2 = sn.ffn_fwd(*fargs)
            assert torch.equal(Y1.view(torch.int16), Y2.view(torch.int16))
        aargs = (inp.Q, inp.K, inp.V, kept_h, dev(inp.ids), masks_dev(inp.masks),
                 dev(inp.sample_table), dev(inp.table_offsets))
        O1 = sn.attend_fwd(*aargs).clone()
        O2 = sn.attend_fwd(*aargs)
        assert torch.equal(O1.view(torch.int16), O2.view(torch.int16))
    assert sn.last_status() == 0


def test_bounded_wait_expires_and_context_survives(sn):
    """A device wait that nothing satisfies gives up after its limit, reports TIMEOUT through the
    status word and frees what it holds; the context then works as before."""
    assert sn.last_status() == 0
    sn.selftest_wait_expiry(100000)
    st = sn.last_status()
    assert st & sentry.STATUS_BIT_TIMEOUT, st
    assert sn.last_status() == 0          # reading clears it
    w = synth.config4().with_(B=6)
    inp = synth.generate(w, n_s_of)
    kept_h, kept_c = parity.gate_lists(sn, inp)
    assert parity.ffn_parity(sn, inp, kept_c) <= TOL["bf16"]
    err, _ = parity.attend_parity(sn, inp, kept_h)
    assert err <= TOL["bf16"]
    with pytest.raises(sentry.SentryError):
        sn.selftest_wait_expiry(0)


def test_ffn_with_weights_materialised_once(sn):
    """sentry_ffn_prepack + sentry_ffn_fwd_packed: the pruned weights are gathered once (Section 4.6)
    and reused; results bit-identical to sentry_ffn_fwd and within tolerance of the oracle."""
    for w in (synth.config1(), synth.config2().with_(B=40), synth.config4().with_(B=24), synth.config5(16, 256)):
        inp = synth.generate(w, n_s_of)
        _, kept_c = parity.gate_lists(sn, inp)
        X, W1, W2 = inp.X.cuda(), inp.W1.cuda(), inp.W2.cuda()
        los, ids, masks = dev(inp.list_of_sample), dev(inp.ids), masks_dev(inp.masks)
        packed = sn.ffn_prepack(W1, W2, kept_c)
        Y_ref = sn.ffn_fwd(X, W1, W2, kept_c, los, ids, masks).clone()
        for _ in range(2):   # the packed buffer is reused
            Y = sn.ffn_fwd_packed(X, packed, w.F, w.k_c, kept_c.shape[0], los, ids, masks)
            assert torch.equal(Y.view(torch.int16 if w.dtype == "bf16" else torch.int32),
                               Y_ref.view(torch.int16 if w.dtype == "bf16" else torch.int32))
        want = oracle.ffn(inp.X, inp.W1, inp.W2, kept_c.cpu().numpy(), inp.list_of_sample, inp.ids, inp.masks)
        got = Y.float().cpu().numpy()
        err = parity.rel_err(got, want, w.dtype, np.ones(got.shape[:2], dtype=bool))
        parity.record(w.name, "ffn_pk", err, parity.raw_rel_err(got, want), "weights materialised once")
        assert err <= TOL[w.dtype]
        assert sn.last_status() == 0
    with pytest.raises(sentry.SentryError) as e:   # buffer too small: refused on the host
        sn.ffn_prepack(W1, W2, kept_c, packed=torch.empty((256,), dtype=torch.uint8, device="cuda"))
    assert e.value.code == -4

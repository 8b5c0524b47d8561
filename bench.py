#!/usr/bin/env python
"""Benchmark of the pruned-layer hot path (gate selection -> sparse GQA attention ->
channel-compacted FFN) through libsentry's C ABI on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4] [--impl ours|reference]

One "step" = one pass of the whole path over one batch of the chosen synthetic
workload.  Prints ONE JSON line (rank 0).  `value` is whole-job present-tokens/s
with inputs resident in HBM; `e2e` is the same through the public API with pinned
host buffers and host<->device copies inside the timed region; `roofline` is the
dominant kernel against the measured peak; `cpu_baseline` is the float64 oracle on
a bounded sample of the same workload on this machine's host cores.

With N > 1 (torchrun) every rank runs the full batch of the workload on its own
GPU (weak scaling, no data-path collective); time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
TABLE_LAYOUT = "auto"   # set from --table-layout
GATE_MULTI = False        # set from --gate-multi
LONG_SELECT = 0           # set from --long-select (SENTRY_OPT_LONG_SELECT)
SEPARATE_GATE = False     # set from --separate-gate
# fp32 FMA peak of the plain ALUs: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (unit counts and max SM clock)
ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu captures (profiles/),
# keyed by (kernel slot, workload); None once the kernel has changed since its capture.
NCU_TRAFFIC = {("attend_core", "cfg4_full_layer"): 41.47e6, ("ffn_main", "cfg4_full_layer"): 36.74e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# --------------------------------------------------------------------------- model
def work_model(w: synth.Workload, masks: np.ndarray, kept_heads: np.ndarray, num_active) -> dict:
    """Algorithmic work of one step: present tokens, useful FLOPs and the bytes each
    kernel has to move (what the method needs, not what a kernel happens to touch)."""
    e = 4 if w.dtype == "f32" else 2
    r = w.Hq // w.Hk
    tokens = 0
    att_flops = ffn_flops = 0.0
    b_score = b_core = b_ffn_rows = 0.0
    n_masks = len(masks)
    for b in range(n_masks):
        tv = synth.present_count(w, int(masks[b]))
        U = num_active(tv)
        G = len(set(int(h) // r for h in kept_heads[b]))
        tokens += tv
        att_flops += w.k_h * (2.0 * tv * U * w.d + 4.0 * U * tv * w.d) + G * tv * w.d
        ffn_flops += 4.0 * w.D * w.k_c * tv
        # score pass: Q of kept heads + K of referenced groups in, one fp32 score per (head, token) out
        b_score += e * w.d * tv * (w.k_h + G) + 4.0 * w.k_h * tv
        # core: K, V of referenced groups + active Q rows + scores in, O of kept heads out
        b_core += e * w.d * tv * (2 * G + w.k_h) + e * w.d * U * w.k_h + 4.0 * w.k_h * tv
        b_ffn_rows += 2.0 * w.D * e * tv
    n_lists = len(set(int(m) for m in masks))
    b_weights = 2.0 * w.D * w.k_c * e * n_lists
    att_bytes = sum(e * w.d * synth.present_count(w, int(masks[b])) *
                    (2 * w.k_h + 2 * len(set(int(h) // r for h in kept_heads[b])))
                    for b in range(n_masks))
    return {"tokens": tokens, "att_flops": att_flops, "ffn_flops": ffn_flops,
            "att_bytes": float(att_bytes),
            "kernel_bytes": {"attend_score": b_score, "attend_core": b_core,
                             "ffn_main": b_ffn_rows + b_weights,
                             "ffn_prepare": 2 * b_weights,
                             "gate_expand": 4.0 * (n_masks * w.k_h + n_lists * w.k_c)},
            "kernel_flops": {"ffn_main": ffn_flops}}


def t_att_all(prof, n_prof):
    """Seconds per step spent in the attention kernels (per-kernel pass)."""
    return sum(prof[k][0] for k in prof if k.startswith("attend")) / n_prof * 1e-3


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# -------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML every 5 ms."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.samples = index, False, []
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception as ex:  # pragma: no cover
            self.err = repr(ex)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                util = nv.nvmlDeviceGetUtilizationRates(self.h).gpu
                self.samples.append((time.time(), sm, int(reasons), util))
            except Exception:
                pass
            time.sleep(0.005)

    def summary(self, t0: float, t1: float) -> dict:
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml_unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1] or \
                 [s for s in self.samples if s[3] >= 50] or self.samples
        bits = 0
        for s in inside:
            bits |= s[2]
        names = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        reasons = [n for b, n in names.items() if bits & b]
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": float(self.max_sm),
                "reasons": reasons, "samples": len(inside)}


# ---------------------------------------------------------------------- distributed
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), \
        int(os.environ.get("WORLD_SIZE", 1))


def aggregate(local_units: float, local_ms: float, device: str):
    """Whole-job units (sum over ranks) and time (max over ranks).  Works on any
    initialised backend (nccl on GPU, gloo on CPU); a no-op without one."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return local_units, local_ms
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()), float(t.item())


def barrier_sync():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
    torch.cuda.synchronize()


# ------------------------------------------------------------------------ reference
def oracle_sample_run(inp: synth.Inputs, sel: np.ndarray, kept_h: np.ndarray, kept_c: np.ndarray):
    """The oracle, as it stands, on the samples `sel` of the workload: gate + attend + ffn."""
    import oracle
    w = inp.w
    masks = inp.masks[sel]
    kh = oracle.gate_select(inp.scores_heads, masks, w.k_h)
    kc = oracle.gate_select(inp.scores_ch, inp.subsets, w.k_c)
    oracle.attend(inp.Q[sel], inp.K[sel], inp.V[sel], kh, inp.ids, masks, c=w.c,
                  sample_table=inp.sample_table, table_offsets=inp.table_offsets)
    oracle.ffn(inp.X[sel], inp.W1, inp.W2, kc, inp.list_of_sample[sel], inp.ids, masks)
    return int(sum(synth.present_count(w, int(m)) for m in masks))


def cpu_sample_inputs(w: synth.Workload, n_max: int):
    """A small CPU batch with the workload's shapes and subset mix (first n_max samples of a
    stratified order), for timing the oracle."""
    import oracle
    wb = w.with_(B=min(w.B, max(n_max, 1)))
    if w.mask_rule == "thirds":  # keep all subsets represented in a short batch
        wb = wb.with_(B=min(w.B, max(n_max, 3)))
    inp = synth.generate(wb, lambda tv: oracle.num_active(tv, w.c))
    return inp


def time_oracle(w: synth.Workload, budget_s: float):
    """Time the oracle, as it stands, on a bounded sample: whole passes over up to 3 x cores
    samples of the workload until about budget_s seconds of wall time have gone.  Returns
    (tokens/s, cores, description)."""
    import oracle
    cores = oracle.threads()
    inp = cpu_sample_inputs(w, 3 * cores)
    sel = np.arange(inp.w.B)
    oracle_sample_run(inp, sel[:1], None, None)  # builds/loads the library outside the timing
    reps, tok = 0, 0
    t0 = time.perf_counter()
    dt = 0.0
    while reps == 0 or (dt < budget_s and reps < 1000):
        tok += oracle_sample_run(inp, sel, None, None)
        reps += 1
        dt = time.perf_counter() - t0
    return tok / dt, cores, "%d samples x %d passes of %s in %.1f s (gate+attend+ffn, float64, OpenMP over samples)" % (
        len(sel), reps, w.name, dt)


def run_reference(args, w: synth.Workload):
    rank, _, world = dist_env()
    if rank != 0:
        return
    import oracle
    cores = oracle.threads()
    total_budget = 150.0
    inp = cpu_sample_inputs(w, 3 * cores)
    t0 = time.perf_counter()
    oracle_sample_run(inp, np.arange(1), None, None)
    t_one = time.perf_counter() - t0
    per_step = total_budget / max(1, args.steps + args.warmup)
    n = int(max(1, min(inp.w.B, (per_step / max(t_one / 1.0, 1e-4)) * min(cores, inp.w.B) // 1)))
    n = max(1, min(n, inp.w.B))
    sel = np.arange(n)
    for _ in range(args.warmup):
        oracle_sample_run(inp, sel, None, None)
    t0 = time.perf_counter()
    tok = 0
    for _ in range(args.steps):
        tok += oracle_sample_run(inp, sel, None, None)
    dt = time.perf_counter() - t0
    val = tok / dt
    line = {"impl": "reference", "metric": "pruned_layer_tokens_per_s", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dt / max(1, args.steps), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sample": "%d samples per step" % n},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": "%d samples of %s per step, %d steps" % (n, w.name, args.steps)},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- ours
class DeviceSet:
    """One resident copy of a step's inputs and outputs."""

    def __init__(self, inp: synth.Inputs, dev: str, src: "DeviceSet" = None):
        w = inp.w
        dt = synth.torch_dtype(w)
        if src is None:
            self.Q, self.K, self.V, self.X = (t.to(dev) for t in (inp.Q, inp.K, inp.V, inp.X))
        else:
            self.Q, self.K, self.V, self.X = (t.clone() for t in (src.Q, src.K, src.V, src.X))
        self.O = torch.empty((w.B, w.k_h, w.T, w.d), dtype=dt, device=dev)
        self.Y = torch.empty((w.B, w.T, w.D), dtype=dt, device=dev)
        self.kept_h = torch.empty((w.B, w.k_h), dtype=torch.int32, device=dev)
        self.kept_c = torch.empty((len(inp.subsets), w.k_c), dtype=torch.int32, device=dev)

    def nbytes(self):
        return sum(t.numel() * t.element_size() for t in (self.Q, self.K, self.V, self.X, self.O, self.Y))


ATTEND_KERNELS = {"auto": 0, "warp": 1, "tcgen05": 2}


class Workbench:
    """One workload resident on one GPU: inputs, rotating buffer sets, the step and its CUDA graphs.

    A step = gate selection for heads -> attention, and gate selection for channels -> weight
    gather -> FFN, the two branches forked on two streams.  With materialise_once the weight gather
    (sentry_ffn_prepack) and the channel gate run once, before the timed region, as Section 4.6
    describes for a fixed set of modality masks and a fixed budget."""

    def __init__(self, sentry, w: synth.Workload, dev: str, local_rank: int, rank: int, overlap: bool,
                 use_graph: bool, attend_kernel: int, materialise_once: bool = False, max_sets: int = 16,
                 lanes: int = 1):
        self.sentry, self.w, self.dev = sentry, w, dev
        # lanes > 1: consecutive steps (independent batches, different buffer sets) are issued on
        # `lanes` streams in turn, each lane with library contexts (scratch) of its own, so that
        # one step's tail and the next step's start may share the GPU
        self.lanes = max(1, lanes)
        self.ctx = []
        for _ in range(self.lanes):
            a = sentry.Sentry(local_rank)
            b = sentry.Sentry(local_rank) if overlap else a
            for c in (a, b):
                c.set_attend_kernel(attend_kernel)
                c.set_option(sentry.OPT_LONG_SELECT, LONG_SELECT)
            self.ctx.append((a, b))
        self.sn, self.sn2 = self.ctx[0]
        self.branches = [torch.cuda.Stream() if overlap else None for _ in range(self.lanes)]
        self.branch = self.branches[0]
        self.lane_streams = [torch.cuda.Stream() for _ in range(self.lanes)] if self.lanes > 1 else []
        self.once = materialise_once
        self.n_s_of = lambda tv: sentry.num_active_queries(tv, w.c)
        inp = synth.generate(w.with_(seed=w.seed + 1000 * rank), self.n_s_of, device=dev)
        self.inp = inp
        self.ids = torch.as_tensor(inp.ids, device=dev)
        self.masks = torch.as_tensor(inp.masks.astype(np.int64).astype(np.int32), device=dev)
        self.subsets = torch.as_tensor(inp.subsets.astype(np.int64).astype(np.int32), device=dev)
        self.los = torch.as_tensor(inp.list_of_sample, device=dev)
        self.sh, self.sc = torch.as_tensor(inp.scores_heads, device=dev), torch.as_tensor(inp.scores_ch, device=dev)
        # the sample tables in the layout the kernels read with one 128-byte access per sample and warp
        # (score_mode 2: entry-major; the same numbers, transposed once here, outside every timed region)
        layout = TABLE_LAYOUT
        if layout == "auto":
            # the bank-friendly order pays where a group's K and V rows sit in shared memory for the whole
            # call (+3 %); kernels that walk K in segments want a query's samples in ascending order
            layout = "arranged" if w.T * (4 * w.d + 20) + 4096 <= 200 * 1024 else "entry"
        self.table_layout = layout
        self.score_mode = 0 if layout == "query" else 2
        tbl_np = synth.entry_major_tables(w, inp.sample_table, inp.table_offsets, self.n_s_of) \
            if layout == "entry" else inp.sample_table
        self.tbl = torch.as_tensor(tbl_np, device=dev)
        if layout == "arranged":   # sentry_sample_table_arrange: entry-major, bank-friendly visiting order
            self.tbl = self.sn.sample_table_arrange(self.ids, self.tbl, torch.as_tensor(inp.table_offsets, device=dev), c=w.c)
        self.offs = torch.as_tensor(inp.table_offsets, device=dev)
        self.W1, self.W2 = inp.W1, inp.W2
        base = DeviceSet(inp, dev)
        self.set_bytes = base.nbytes()
        self.n_sets = 1 if self.set_bytes >= 2 * L2_BYTES else int(min(max_sets, -(-2 * L2_BYTES // self.set_bytes)))
        self.n_sets = -(-self.n_sets // self.lanes) * self.lanes   # set j always runs on lane j % lanes
        self.sets = [base] + [DeviceSet(inp, dev, base) for _ in range(self.n_sets - 1)]
        self.launches = 0
        self.packed = None
        if self.once:
            self.sn2.gate_select(self.sc, self.subsets, w.k_c, kept=base.kept_c)
            self.packed = self.sn2.ffn_prepack(self.W1, self.W2, base.kept_c)
        for lane in range(self.lanes):               # sizes the workspaces before any capture
            self.step(self.sets[lane], count=True, lane=lane)
        torch.cuda.synchronize()
        assert self.status() == 0, "device status word set during warm-up"
        self.graphs = None
        if use_graph:
            self.graphs = []
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for j, s_ in enumerate(self.sets):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        self.step(s_, lane=j % self.lanes)
                    self.graphs.append(g)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()

    def ffn_branch(self, s: DeviceSet, ctx, gated=False):
        w = self.w
        if gated:
            ctx.ffn_fwd(s.X, self.W1, self.W2, s.kept_c, self.los, self.ids, self.masks, Y=s.Y)
            return ctx.last_launch_count()
        if self.once:
            ctx.ffn_fwd_packed(s.X, self.packed, w.F, w.k_c, len(self.inp.subsets), self.los, self.ids, self.masks, Y=s.Y)
            return ctx.last_launch_count()
        ctx.gate_select(self.sc, self.subsets, w.k_c, kept=s.kept_c)
        n = ctx.last_launch_count()
        ctx.ffn_fwd(s.X, self.W1, self.W2, s.kept_c, self.los, self.ids, self.masks, Y=s.Y)
        return n + ctx.last_launch_count()

    def step(self, s: DeviceSet, count=False, fork=True, lane=0):
        w = self.w
        sn, sn2 = self.ctx[lane]
        branch = self.branches[lane]
        n = 0
        two = fork and branch is not None
        multi = GATE_MULTI and not self.once
        if multi:   # heads and channels selected by one launch, ahead of the fork
            sn.gate_select_multi([(self.sh, self.masks, w.k_h, 0, s.kept_h), (self.sc, self.subsets, w.k_c, 0, s.kept_c)])
            n += sn.last_launch_count()
        if two:
            cur = torch.cuda.current_stream()
            branch.wait_stream(cur)
            with torch.cuda.stream(branch):
                n += self.ffn_branch(s, sn2, gated=multi)
        if not multi and not SEPARATE_GATE:
            # head selection and attention in one call (one launch where K and V of a group fit in shared memory)
            sn.gate_attend_fwd(self.sh, w.k_h, s.Q, s.K, s.V, self.ids, self.masks, self.tbl, self.offs, c=w.c,
                               score_mode=self.score_mode, O=s.O, kept_heads=s.kept_h)
            n += sn.last_launch_count()
        else:
            if not multi:
                sn.gate_select(self.sh, self.masks, w.k_h, kept=s.kept_h)
                n += sn.last_launch_count()
            sn.attend_fwd(s.Q, s.K, s.V, s.kept_h, self.ids, self.masks, self.tbl, self.offs, c=w.c, O=s.O,
                          score_mode=self.score_mode)
            n += sn.last_launch_count()
        if two:
            torch.cuda.current_stream().wait_stream(branch)
        else:
            n += self.ffn_branch(s, sn, gated=multi)
        if count:
            self.launches = n

    def run_steps(self, n, start=0):
        if self.lanes == 1:
            for i in range(n):
                if self.graphs is not None:
                    self.graphs[(start + i) % self.n_sets].replay()
                else:
                    self.step(self.sets[(start + i) % self.n_sets])
            return
        cur = torch.cuda.current_stream()
        for ls in self.lane_streams:
            ls.wait_stream(cur)
        for i in range(n):
            j = (start + i) % self.n_sets
            with torch.cuda.stream(self.lane_streams[j % self.lanes]):
                if self.graphs is not None:
                    self.graphs[j].replay()
                else:
                    self.step(self.sets[j], lane=j % self.lanes)
        for ls in self.lane_streams:
            cur.wait_stream(ls)

    def time_blocks(self, steps: int, replays: int, warmup: int):
        """`replays` blocks of `steps` steps each, every block bracketed by a barrier and a device
        synchronisation on both sides and timed with CUDA events.  Returns the per-block ms."""
        self.run_steps(max(3, warmup))
        out = []
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for r in range(replays):
            barrier_sync()
            ev0.record()
            self.run_steps(steps, start=r * steps)
            ev1.record()
            barrier_sync()
            out.append(ev0.elapsed_time(ev1))
        return out

    def per_kernel(self, n_prof: int):
        """Per-kernel CUDA-event pass (one stream, no graph): {kernel: (total ms, launches)}."""
        sn = self.sn
        sn.profile_enable(True)
        for i in range(3):
            self.step(self.sets[i % self.n_sets], fork=False)
        sn.profile_read()
        for i in range(n_prof):
            self.step(self.sets[i % self.n_sets], fork=False)
        prof = sn.profile_read()
        sn.profile_enable(False)
        return prof

    def time_chained_layer(self, steps: int, replays: int):
        """The full pruned encoder layer chained on one stream: gate selection for heads -> pruned Q/K/V
        projections of X -> SentryAttend -> pruned output projection -> gate selection for channels ->
        channel-compacted FFN on the projected rows (no residual or normalisation: the paper names none).
        Returns (median ms per step, launches per step)."""
        w, sn, dev = self.w, self.sn, self.dev
        if w.D % 8 != 0:
            return None
        dt = synth.torch_dtype(w)
        g = torch.Generator(device=dev).manual_seed(w.seed + 77)
        mk = lambda *shape: (torch.randn(shape, generator=g, device=dev) * (4 * w.w_std)).to(dt)
        WQ, WK, WV, WO = mk(w.D, w.Hq * w.d), mk(w.D, w.Hk * w.d), mk(w.D, w.Hk * w.d), mk(w.Hq * w.d, w.D)
        s0 = self.sets[0]
        Q, K, V = torch.zeros_like(s0.Q), torch.zeros_like(s0.K), torch.zeros_like(s0.V)
        H = torch.empty_like(s0.X)
        n = [0]

        def chain(count=False):
            c = 0
            sn.gate_select(self.sh, self.masks, w.k_h, kept=s0.kept_h); c += sn.last_launch_count()
            sn.project_qkv(s0.X, WQ, WK, WV, s0.kept_h, self.ids, self.masks, w.Hq, w.Hk, w.d, Q=Q, K=K, V=V)
            c += sn.last_launch_count()
            sn.attend_fwd(Q, K, V, s0.kept_h, self.ids, self.masks, self.tbl, self.offs, c=w.c, O=s0.O,
                          score_mode=self.score_mode)
            c += sn.last_launch_count()
            sn.project_out(s0.O, WO, s0.kept_h, self.ids, self.masks, w.Hq, out=H); c += sn.last_launch_count()
            sn.gate_select(self.sc, self.subsets, w.k_c, kept=s0.kept_c); c += sn.last_launch_count()
            sn.ffn_fwd(H, self.W1, self.W2, s0.kept_c, self.los, self.ids, self.masks, Y=s0.Y)
            c += sn.last_launch_count()
            if count:
                n[0] = c

        chain(count=True)
        torch.cuda.synchronize()
        graph = None
        if self.graphs is not None:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    chain()
            torch.cuda.current_stream().wait_stream(side)
        run = graph.replay if graph is not None else chain
        for _ in range(3):
            run()
        out = []
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(replays):
            torch.cuda.synchronize()
            ev0.record()
            for _ in range(steps):
                run()
            ev1.record()
            torch.cuda.synchronize()
            out.append(ev0.elapsed_time(ev1) / steps)
        assert sn.last_status() == 0
        return float(np.median(out)), n[0]

    def work(self):
        kept_h_host = self.sets[0].kept_h.cpu().numpy()
        return work_model(self.w, self.inp.masks, kept_h_host, self.n_s_of)

    def status(self):
        st = 0
        for a, b in self.ctx:
            st |= a.last_status() | b.last_status()
        return st

    def close(self):
        for a, b in self.ctx:
            if b is not a:
                b.close()
            a.close()
        self.graphs = None
        self.sets = None
        torch.cuda.empty_cache()


def stage_fractions(wm, prof, n_prof, peaks):
    t_att = sum(prof[k][0] for k in prof if k.startswith("attend")) / n_prof * 1e-3
    t_ffn = sum(prof[k][0] for k in prof if k.startswith("ffn")) / n_prof * 1e-3
    t_main = prof["ffn_main"][0] / n_prof * 1e-3 if "ffn_main" in prof else t_ffn
    return {
        "attend": {"ms": t_att * 1e3, "hbm_frac": wm["att_bytes"] / max(t_att, 1e-12) / 1e9 / peaks["hbm_gbs"],
                   "useful_tflops": wm["att_flops"] / max(t_att, 1e-12) / 1e12},
        "ffn": {"ms": t_ffn * 1e3,
                "tensor_frac": wm["ffn_flops"] / max(t_ffn, 1e-12) / 1e12 / peaks["bf16_tflops"],
                "main_kernel_tensor_frac": wm["ffn_flops"] / max(t_main, 1e-12) / 1e12 / peaks["bf16_tflops"],
                "useful_tflops": wm["ffn_flops"] / max(t_ffn, 1e-12) / 1e12}}


def quick_moe(sentry, dev: str, local_rank: int, peaks):
    """The Sparse-MoE block (Section 4.6) on a synthetic shape of its own (the paper gives none): 32 768 tokens,
    d_model 256, 8 experts of d_ff 1024 pruned to 512 channels each, top-2 routing with skewed expert popularity.
    Median of 5 blocks of 20 calls on rotating inputs; weights gathered per call, and materialised once."""
    N, D, F, E, top_k, k_c = 32768, 256, 1024, 8, 2, 512
    m = synth.generate_moe(N, D, F, E, top_k, k_c, "bf16", seed=11, skew=1.0, device=dev)
    sn = sentry.Sentry(local_rank)
    kept = torch.as_tensor(m.kept, device=dev)
    ids = torch.as_tensor(m.expert_ids, device=dev)
    wts = torch.as_tensor(m.expert_weights, device=dev)
    n_sets = 8   # 8 x (X + Y) = 268 MB of rotating activations (> L2) beside the 8 MB of expert weights
    Xs = [m.X] + [torch.randn_like(m.X, dtype=torch.float32).to(m.X.dtype) for _ in range(n_sets - 1)]
    Ys = [torch.empty_like(m.X) for _ in range(n_sets)]
    packed = sn.moe_prepack(m.W1, m.W2, kept)
    out = {"workload": "moe_N32768_D256_F1024_E8_top2_kc512", "tokens": N}

    def run(i, once):
        if once:
            sn.moe_ffn_fwd(Xs[i % n_sets], ids, wts, packed=packed, F=F, E=E, k_c=k_c, Y=Ys[i % n_sets])
        else:
            sn.moe_ffn_fwd(Xs[i % n_sets], ids, wts, W1=m.W1, W2=m.W2, kept_channels=kept, Y=Ys[i % n_sets])

    flops = 4.0 * D * k_c * N * top_k
    for once in (False, True):
        for i in range(5):
            run(i, once)
        launches = sn.last_launch_count()
        torch.cuda.synchronize()
        blocks = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for r in range(5):
            e0.record()
            for i in range(20):
                run(r * 20 + i, once)
            e1.record()
            torch.cuda.synchronize()
            blocks.append(e0.elapsed_time(e1) / 20)
        ms = float(np.median(blocks))
        key = "materialised_once" if once else "per_call_gather"
        out[key] = {"ms_per_call": ms, "tokens_per_s": N / (ms * 1e-3), "launches_per_call": launches,
                    "tensor_frac": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
    out["device_status"] = sn.last_status()
    sn.close()
    return out


def quick_fp8_ffn(sentry, dev: str, local_rank: int, peaks):
    """The FFN of workload 3 (65 536 rows, d_model 256, 512 of 1024 channels kept, one list) and of workload 4
    (43 520 present rows, d_model 384, 614 of 1536 channels kept, three lists) with FP8 e4m3 operands
    (sentry_ffn_fwd_fp8, weights prepacked once) beside the same call in bf16 (sentry_ffn_fwd_packed):
    median of 5 blocks of 20 calls on rotating inputs larger than L2.  FLOPs as for bf16: 4 D k_c per row."""
    sn = sentry.Sentry(local_rank)
    out = {}
    for key, w in (("cfg3", synth.config3()), ("cfg4", synth.config4())):
        rng = np.random.default_rng(5)
        inp = synth.generate(w, lambda tv: sentry.num_active_queries(tv, w.c), tensors=False)
        n_lists = len(inp.subsets)
        kept = torch.as_tensor(np.stack([np.sort(rng.permutation(w.F)[:w.k_c]) for _ in range(n_lists)]).astype(np.int32),
                               device=dev)
        los = torch.as_tensor(inp.list_of_sample, device=dev)
        ids = torch.as_tensor(inp.ids, device=dev)
        masks = torch.as_tensor(inp.masks.astype(np.int64).astype(np.int32), device=dev)
        rows = int(sum(synth.present_count(w, int(m)) for m in inp.masks))
        n_sets = 8
        Xb = [torch.randn((w.B, w.T, w.D), device=dev).to(torch.bfloat16) for _ in range(n_sets)]
        Xq = [(x.float() * 100.0).to(torch.float8_e4m3fn).view(torch.uint8) for x in Xb]
        W1 = (torch.randn((w.D, w.F), device=dev) * 0.02).to(torch.bfloat16)
        W2 = (torch.randn((w.F, w.D), device=dev) * 0.02).to(torch.bfloat16)
        W1q = (W1.float() * 5000.0).to(torch.float8_e4m3fn).view(torch.uint8)
        W2q = (W2.float() * 5000.0).to(torch.float8_e4m3fn).view(torch.uint8)
        Y = [torch.empty((w.B, w.T, w.D), dtype=torch.bfloat16, device=dev) for _ in range(n_sets)]
        p16 = sn.ffn_prepack(W1, W2, kept)
        p8 = sn.ffn_prepack_e4m3(W1q, W2q, kept)
        flops = 4.0 * w.D * w.k_c * rows
        res = {"workload": "ffn of %s (%d present rows, D=%d, k_c=%d, %d lists), weights materialised once"
                           % (w.name, rows, w.D, w.k_c, n_lists)}
        for name in ("bf16", "fp8_e4m3"):
            def run(i):
                if name == "bf16":
                    sn.ffn_fwd_packed(Xb[i % n_sets], p16, w.F, w.k_c, n_lists, los, ids, masks, Y=Y[i % n_sets])
                else:
                    sn.ffn_fwd_fp8(Xq[i % n_sets], p8, w.F, w.k_c, n_lists, 0.01, 2e-4, 2e-4, 0.01, los, ids, masks,
                                   Y=Y[i % n_sets])
            for i in range(5):
                run(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            blocks = []
            for r in range(5):
                e0.record()
                for i in range(20):
                    run(r * 20 + i)
                e1.record()
                torch.cuda.synchronize()
                blocks.append(e0.elapsed_time(e1) / 20)
            ms = float(np.median(blocks))
            res[name] = {"ms_per_call": ms, "tokens_per_s": rows / (ms * 1e-3), "tflops": flops / (ms * 1e-3) / 1e12,
                         "frac_of_bf16_peak": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
            if name == "fp8_e4m3":
                # peak of its own operand type: the measured bf16 figure x the nominal 8-bit : 16-bit ratio (2)
                res[name]["frac_of_fp8_peak"] = res[name]["frac_of_bf16_peak"] / 2.0
        if key == "cfg3":
            out.update(res)          # the first shape keeps its place at the top level of the object
        else:
            out[key] = res
        del Xb, Xq, Y
        torch.cuda.empty_cache()
    out["device_status"] = sn.last_status()
    sn.close()
    return out


def quick_config(sentry, name: str, dev: str, local_rank: int, peaks, args):
    """Short measurement of one other workload for the `configs` table: median of 3 blocks of at
    least ~10 ms, plus the per-kernel pass."""
    w = synth.by_name(name)
    wb = Workbench(sentry, w, dev, local_rank, 0, not args.no_overlap, not args.no_graph,
                   ATTEND_KERNELS[args.attend_kernel], max_sets=8, lanes=args.lanes)
    wm = wb.work()
    probe = wb.time_blocks(5, 1, 3)[0] / 5
    steps = int(max(5, min(400, 10.0 / max(probe, 1e-3))))
    blocks = wb.time_blocks(steps, 3, 3)
    ms = float(np.median(blocks)) / steps
    prof = wb.per_kernel(min(steps, 20))
    st = stage_fractions(wm, prof, min(steps, 20), peaks)
    out = {"workload": w.name, "tokens_per_s": wm["tokens"] / (ms * 1e-3), "ms_per_step": ms, "steps_per_block": steps,
           "present_tokens": wm["tokens"], "attend_ms": st["attend"]["ms"], "attend_hbm_frac": st["attend"]["hbm_frac"],
           "ffn_ms": st["ffn"]["ms"], "ffn_tensor_frac": st["ffn"]["tensor_frac"],
           "ffn_main_tensor_frac": st["ffn"]["main_kernel_tensor_frac"],
           "useful_tflops": (wm["att_flops"] + wm["ffn_flops"]) / (ms * 1e-3) / 1e12, "device_status": wb.status()}
    wb.close()
    return out


def run_ours(args, w: synth.Workload):
    import paper_2604_08971_b200 as sentry
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libsentry has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    sentry.build()
    sampler = ClockSampler(local_rank)
    sampler.start()

    wb = Workbench(sentry, w, dev, local_rank, rank, not args.no_overlap, not args.no_graph,
                   ATTEND_KERNELS[args.attend_kernel], lanes=args.lanes)
    sn, inp, base = wb.sn, wb.inp, wb.sets[0]
    n_sets, set_bytes = wb.n_sets, wb.set_bytes

    # ---- device-resident timing: `replays` blocks of exactly `steps` steps, median block
    t_wall0 = time.time()
    blocks = wb.time_blocks(args.steps, args.replays, args.warmup)
    t_wall1 = time.time()
    local_ms = float(np.median(blocks))
    wm = wb.work()
    total_tokens, ms = aggregate(float(wm["tokens"]) * args.steps, local_ms, dev)
    clocks = sampler.summary(t_wall0, t_wall1)

    # ---- per-kernel pass (same steps, events around every kernel, no graph)
    n_prof = min(args.steps, 50)
    prof = wb.per_kernel(n_prof)

    # ---- the whole layer chained X -> Q,K,V -> attention -> output projection -> FFN
    chained = None
    if world == 1 and not args.no_once:
        res = wb.time_chained_layer(max(5, args.steps // 4), 3)
        if res is not None:
            c_ms, c_launches = res
            r_ = w.Hq // w.Hk
            proj_flops = sum(2.0 * w.D * w.d * synth.present_count(w, int(m)) *
                             (2 * w.k_h + 2 * len(set(int(h) // r_ for h in kh)))
                             for m, kh in zip(inp.masks, base.kept_h.cpu().numpy()))
            chained = {"ms_per_step": c_ms, "tokens_per_s": wm["tokens"] / (c_ms * 1e-3), "gpu_launches_per_step": c_launches,
                       "useful_tflops": (wm["att_flops"] + wm["ffn_flops"] + proj_flops) / (c_ms * 1e-3) / 1e12,
                       "projection_flops": proj_flops,
                       "what": "one stream: gate(heads), sentry_project_qkv, sentry_attend_fwd, sentry_project_out, "
                               "gate(channels), sentry_ffn_fwd on the projected rows"}

    # ---- the same step with the pruned FFN weights materialised once (Section 4.6)
    once = None
    if world == 1 and not args.no_once:
        wb1 = Workbench(sentry, w, dev, local_rank, rank, not args.no_overlap, not args.no_graph,
                        ATTEND_KERNELS[args.attend_kernel], materialise_once=True, lanes=args.lanes)
        b1 = wb1.time_blocks(args.steps, max(3, args.replays // 2 + 1), args.warmup)
        ms1 = float(np.median(b1)) / args.steps
        once = {"value": wm["tokens"] / (ms1 * 1e-3), "unit": "tokens/s", "ms_per_step": ms1,
                "gpu_launches_per_step": wb1.launches,
                "what": "channel gate selection and weight gather (sentry_ffn_prepack) run once before the timed "
                        "region; a step = head gate selection + attention + sentry_ffn_fwd_packed"}
        wb1.close()

    # ---- two steps in flight: consecutive steps (independent batches on different buffer sets) issued on two
    # streams in turn, each with library contexts of its own, so that the ragged end of one step's launches and
    # the start of the next share the GPU.  Reported beside the headline, which runs one step at a time.
    overlapped = None
    if world == 1 and not args.no_once and args.lanes == 1:
        wb2 = Workbench(sentry, w, dev, local_rank, rank, not args.no_overlap, not args.no_graph,
                        ATTEND_KERNELS[args.attend_kernel], lanes=2)
        b2 = wb2.time_blocks(args.steps, max(3, args.replays // 2 + 1), args.warmup)
        ms2 = float(np.median(b2)) / args.steps
        overlapped = {"value": wm["tokens"] / (ms2 * 1e-3), "unit": "tokens/s", "ms_per_step": ms2, "steps_in_flight": 2,
                      "device_status": wb2.status(),
                      "what": "the same steps, issued alternately on two streams (two independent batches in flight); "
                              "ms_per_step = block time / steps"}
        wb2.close()

    # ---- end to end: pinned host buffers in, results out, every step
    ids, masks, subsets, los, sh, sc, tbl, offs, W1, W2 = (wb.ids, wb.masks, wb.subsets, wb.los, wb.sh, wb.sc,
                                                           wb.tbl, wb.offs, wb.W1, wb.W2)
    host_in = [t.cpu().pin_memory() for t in (base.Q, base.K, base.V, base.X)]
    small_in = [t.cpu().pin_memory() for t in (ids, masks, subsets, los, sh, sc, tbl, offs, W1, W2)]
    host_out = [torch.empty_like(base.O, device="cpu").pin_memory(),
                torch.empty_like(base.Y, device="cpu").pin_memory()]
    dsmall = [ids, masks, subsets, los, sh, sc, tbl, offs, W1, W2]
    h2d = sum(t.numel() * t.element_size() for t in host_in + small_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)

    # The batch goes through in chunks of samples on three streams, so that the upload of chunk
    # i+1, the kernels of chunk i and the download of chunk i-1 overlap (samples are independent).
    n_chunks = int(max(1, min(8, w.B // 16, h2d // (32 << 20))))   # ~32 MB of input per chunk
    bounds = [(w.B * i) // n_chunks for i in range(n_chunks + 1)]
    s_up, s_down = torch.cuda.Stream(), torch.cuda.Stream()
    kept_c_e2e = torch.empty_like(base.kept_c)

    def e2e_steps(n):
        """n steps, pipelined across chunks AND steps: chunk i of step s+1 is uploaded once the
        kernels of chunk i of step s have read their inputs, and its kernels start once chunk i's
        results of step s have left for the host.  Every step uploads all inputs and downloads all
        results; only the order of independent copies and kernels overlaps."""
        cur = torch.cuda.current_stream()
        s_up.wait_stream(cur)
        s_down.wait_stream(cur)
        k_done = [None] * n_chunks
        d_done = [None] * n_chunks
        for _ in range(n):
            ups = []
            with torch.cuda.stream(s_up):
                if k_done[-1] is not None:
                    s_up.wait_event(k_done[-1])      # the small inputs are read by every chunk's kernels
                for dst, src in zip(dsmall, small_in):
                    dst.copy_(src, non_blocking=True)
                for i in range(n_chunks):
                    b0, b1 = bounds[i], bounds[i + 1]
                    for dst, src in zip((base.Q, base.K, base.V, base.X), host_in):
                        dst[b0:b1].copy_(src[b0:b1], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(s_up)
                    ups.append(ev)
            for i in range(n_chunks):
                b0, b1 = bounds[i], bounds[i + 1]
                cur.wait_event(ups[i])
                if d_done[i] is not None:
                    cur.wait_event(d_done[i])        # O / Y of this chunk are about to be overwritten
                sn.gate_attend_fwd(sh, w.k_h, base.Q[b0:b1], base.K[b0:b1], base.V[b0:b1], ids, masks[b0:b1], tbl, offs,
                                   c=w.c, score_mode=wb.score_mode, O=base.O[b0:b1], kept_heads=base.kept_h[b0:b1])
                sn.gate_select(sc, subsets, w.k_c, kept=kept_c_e2e)
                sn.ffn_fwd(base.X[b0:b1], W1, W2, kept_c_e2e, los[b0:b1], ids, masks[b0:b1], Y=base.Y[b0:b1])
                k_done[i] = torch.cuda.Event()
                k_done[i].record(cur)
                s_down.wait_event(k_done[i])
                with torch.cuda.stream(s_down):
                    host_out[0][b0:b1].copy_(base.O[b0:b1], non_blocking=True)
                    host_out[1][b0:b1].copy_(base.Y[b0:b1], non_blocking=True)
                    d_done[i] = torch.cuda.Event()
                    d_done[i].record(s_down)
        cur.wait_stream(s_down)
        cur.wait_stream(s_up)

    n_e2e = max(3, min(args.steps, 20))
    e2e_tokens, e2e_ms = None, None
    if not args.no_e2e:
        e2e_steps(3)
        barrier_sync()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        e2e_steps(n_e2e)
        ev1.record()
        barrier_sync()
        e2e_tokens, e2e_ms = aggregate(float(wm["tokens"]) * n_e2e, ev0.elapsed_time(ev1), dev)
        torch.cuda.synchronize()
        # what reached the host is what the device holds (outside the timed region)
        if not (torch.equal(host_out[0], base.O.cpu()) and torch.equal(host_out[1], base.Y.cpu())):
            raise RuntimeError("end-to-end leg: host results differ from the device buffers")
    status = wb.status()
    launches = wb.launches
    graphs_on = wb.graphs is not None
    two_streams = wb.branch is not None
    host_in = small_in = host_out = None
    wb.close()

    if rank != 0:
        sampler.stop_flag = True
        return
    peaks, peak_kind = load_peaks()
    # dominant kernel = largest share of the per-kernel pass
    per_kernel = {k: {"ms_per_launch": v[0] / v[1], "launches_per_step": v[1] / n_prof,
                      "share": v[0] / max(1e-9, sum(x[0] for x in prof.values()))}
                  for k, v in prof.items()}
    top = max(prof, key=lambda k: prof[k][0])
    t_launch = prof[top][0] / prof[top][1] * 1e-3
    if "attend_score" not in prof:
        # single-kernel attention: it reads Q (kept heads), K, V once and writes O once
        wm["kernel_bytes"]["attend_core"] = wm["att_bytes"]
    if top == "ffn_main":
        fl = wm["kernel_flops"]["ffn_main"]
        by = wm["kernel_bytes"]["ffn_main"]
        t_tensor, t_hbm = fl / (peaks["bf16_tflops"] * 1e12), by / (peaks["hbm_gbs"] * 1e9)
        if t_tensor >= t_hbm and w.dtype in ("bf16", "f16"):
            roof = {"bound": "tensor", "achieved": fl / t_launch / 1e12, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s"}
        else:
            roof = {"bound": "hbm", "achieved": by / t_launch / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        by = wm["kernel_bytes"].get(top, 0.0)
        roof = {"bound": "hbm", "achieved": by / t_launch / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    if top.startswith("attend"):
        # the attention kernels are HBM-bound by their bytes but spend their time in the sampled-score
        # arithmetic on the plain ALUs: report that rate too
        roof["alu_tflops"] = wm["att_flops"] / max(t_att_all(prof, n_prof), 1e-12) / 1e12
        roof["alu_peak_tflops"] = ALU_PEAK_TFLOPS
        roof["alu_frac"] = roof["alu_tflops"] / ALU_PEAK_TFLOPS
    roof.update({"kernel": top, "frac": roof["achieved"] / roof["peak"],
                 "traffic": NCU_TRAFFIC.get((top, w.name)),
                 "peak_source": "%s (burst figure: the kernel is timed alone in the per-kernel pass)" % peak_kind,
                 "ms_per_launch": t_launch * 1e3})
    stages = stage_fractions(wm, prof, n_prof, peaks)

    # ---- the other named workloads and the sweep cells, each measured briefly in this same run
    table = {}
    if world == 1 and not args.no_configs:
        names = ["2", "3a", "3b", "3c", "4"] + ["5:%dx%d" % bt for bt in synth.CONFIG5_CELLS] + ["3b:f16", "4:f16"]
        for name in names:
            try:
                table[name] = quick_config(sentry, name, dev, local_rank, peaks, args)
            except Exception as ex:   # a cell that does not fit or fails must not take the line down
                table[name] = {"error": repr(ex)[:200]}
        try:
            table["moe"] = quick_moe(sentry, dev, local_rank, peaks)
        except Exception as ex:
            table["moe"] = {"error": repr(ex)[:200]}
        try:
            table["ffn_fp8"] = quick_fp8_ffn(sentry, dev, local_rank, peaks)
        except Exception as ex:
            table["ffn_fp8"] = {"error": repr(ex)[:200]}
    sampler.stop_flag = True

    cpu = {"value": None, "unit": "tokens/s", "cores": None, "kind": "oracle", "sample": "skipped"}
    if world == 1 and not args.no_cpu:
        v, cores, what = time_oracle(w, args.cpu_budget)
        cpu = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": what}

    value = total_tokens / (ms * 1e-3)
    line = {
        "metric": "pruned_layer_tokens_per_s", "value": value, "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "batch_per_gpu": w.B, "seq_len": w.T, "modalities": w.M,
                   "d_model": w.D, "q_heads": w.Hq, "kv_heads": w.Hk, "head_dim": w.d, "d_ff": w.F,
                   "kept_heads": w.k_h, "kept_channels": w.k_c, "mask_rule": w.mask_rule,
                   "present_tokens_per_step_per_gpu": wm["tokens"], "parallelism": "replicas x%d" % world,
                   "l2_policy": "rotating %d resident buffer sets, %.0f MB in total (> 126 MB L2)"
                                % (n_sets, n_sets * set_bytes / 1e6),
                   "cuda_graph": graphs_on,
                   "steps_in_flight": args.lanes,
                   "streams": "attention branch and FFN branch forked inside the step" if two_streams
                              else "one stream",
                   "attend_kernel": args.attend_kernel,
                   "sample_table_layout": {"arranged": "sentry_sample_table_arrange, once, outside the timed region (score_mode 2)",
                                           "entry": "entry-major (score_mode 2), transposed once outside the timed region",
                                           "query": "query-major (score_mode 0)"}[wb.table_layout],
                   "step_includes": "gate selection for heads and channels, attention, FFN weight gather and FFN, "
                                    "every step (see materialised_once for the weights gathered once); heads are selected "
                                    + ("by a launch of their own" if args.separate_gate or args.gate_multi else
                                       "through sentry_gate_attend_fwd (inside the attention launch where K/V of a group fit in shared memory)"),
                   "timing": "median of %d blocks of %d steps, each block bracketed by barrier + synchronise "
                             "and timed with CUDA events" % (args.replays, args.steps)},
        "block_ms": blocks, "replays": args.replays,
        "useful_tflops": (wm["att_flops"] + wm["ffn_flops"]) * world * args.steps / (ms * 1e-3) / 1e12,
        "materialised_once": once, "two_steps_in_flight": overlapped, "chained_layer": chained,
        "e2e": None if e2e_ms is None else {"value": e2e_tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": n_e2e,
                "pipeline": "%d sample chunks; upload, kernels and download on three streams, consecutive steps overlapping chunk by chunk" % n_chunks},
        "gpu_launches": launches * args.steps,
        "clocks": clocks, "roofline": roof, "stages": stages, "kernels": per_kernel,
        "configs": table,
        "cpu_baseline": cpu, "device_status": status,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="4",
                    help="1, 2, 3a|3b|3c, 4 (default: the full pruned encoder layer), 5:BxT")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-overlap", action="store_true",
                    help="run the attention branch and the FFN branch of a step on one stream")
    ap.add_argument("--no-cpu", action="store_true", help="skip the timed CPU oracle baseline")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the table of the other named workloads and sweep cells")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg (for profiler launch lists)")
    ap.add_argument("--no-once", action="store_true", help="skip the materialised-once leg (for profiler launch lists)")
    ap.add_argument("--replays", type=int, default=5, help="timed blocks of --steps steps; the median is reported")
    ap.add_argument("--attend-kernel", default="auto", choices=sorted(ATTEND_KERNELS),
                    help="SENTRY_OPT_ATTEND_KERNEL for the attention call")
    ap.add_argument("--long-select", default="auto", choices=["auto", "query-blocks", "per-group"],
                    help="SENTRY_OPT_LONG_SELECT: form of the score + selection step for sequences whose K/V do not fit in shared memory")
    ap.add_argument("--separate-gate", action="store_true",
                    help="sentry_gate_select + sentry_attend_fwd instead of sentry_gate_attend_fwd")
    ap.add_argument("--gate-multi", action="store_true",
                    help="select heads and channels with one sentry_gate_select_multi launch ahead of the fork")
    ap.add_argument("--table-layout", default="auto", choices=["auto", "arranged", "entry", "query"],
                    help="sample tables handed to sentry_attend_fwd: prepared once by sentry_sample_table_arrange "
                         "(score_mode 2), plainly transposed (score_mode 2), or query-major as generated (score_mode 0); "
                         "auto: arranged where K and V of a group fit in shared memory, transposed otherwise; "
                         "the sampled sets are the same")
    ap.add_argument("--lanes", type=int, default=1,
                    help="streams that consecutive steps are issued on in turn (independent batches; 1 = one step at a time)")
    ap.add_argument("--side", default=None, choices=["moe", "ffn_fp8"],
                    help="run only this side measurement of the configs table and print its object (for profiler captures)")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    global TABLE_LAYOUT, GATE_MULTI, LONG_SELECT, SEPARATE_GATE
    SEPARATE_GATE = args.separate_gate
    LONG_SELECT = {"auto": 0, "query-blocks": 1, "per-group": 2}[args.long_select]
    TABLE_LAYOUT = args.table_layout
    GATE_MULTI = args.gate_multi
    w = synth.by_name(args.config)
    if args.side is not None:
        import paper_2604_08971_b200 as sentry
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: libsentry has no CPU fallback")
        sentry.build()
        torch.cuda.set_device(0)
        peaks, _ = load_peaks()
        fn = {"moe": quick_moe, "ffn_fp8": quick_fp8_ffn}[args.side]
        print(json.dumps({args.side: fn(sentry, "cuda:0", 0, peaks)}))
        return
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)
        import torch.distributed as dist
        if dist.is_available() and dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Seeded synthetic inputs for the pruned-layer path.

This module only draws numbers and describes shapes.  It holds none of the
method's arithmetic: the number of sampled keys per query is passed in by the
caller (who asks either the oracle or the CUDA library for it), and nothing
here selects, scores or multiplies anything.  Both the oracle-side tests and
the CUDA-side benchmark import it; it imports neither of them.

The five workloads stand in for the paper's multimodal time-series windows
(wearable and physiological sensor streams through a transformer encoder);
the paper's datasets and trained weights are not reproduced.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Callable, Dict, List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                 # "f32" | "bf16"
    B: int
    lengths: tuple             # tokens per modality, concatenated in id order
    D: int
    Hq: int
    Hk: int
    d: int
    F: int
    k_h: int
    k_c: int
    mask_rule: str             # "all" | "dropout0.3" | "thirds" | "cycle7"
    seed: int
    act_std: float = 1.0       # Q, K, V (and X unless x_std given)
    w_std: float = 0.02
    x_std: Optional[float] = None
    c: int = 5

    @property
    def M(self) -> int:
        return len(self.lengths)

    @property
    def T(self) -> int:
        return int(sum(self.lengths))

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def keep_count(ratio: float, n: int) -> int:
    """Keep ratio -> integer budget: max(1, floor(ratio * n))."""
    return max(1, int(np.floor(ratio * n + 1e-9)))


def split_even(T: int, M: int) -> tuple:
    """T tokens over M modalities; the first T mod M modalities get one more."""
    base, extra = divmod(T, M)
    return tuple(base + (1 if j < extra else 0) for j in range(M))


def config1() -> Workload:
    return Workload("cfg1_tiny_fp32", "f32", 2, (16, 16), 64, 4, 2, 16, 256, 3, 128,
                    "all", 0, act_std=1.0, w_std=0.02, x_std=0.02)


def config2() -> Workload:
    return Workload("cfg2_wearable", "bf16", 256, (64, 64, 64), 128, 8, 2, 16, 512,
                    keep_count(0.5, 8), keep_count(0.5, 512), "dropout0.3", 1)


def config3(head_keep: float = 0.5) -> Workload:
    return Workload("cfg3_physio_kh%d" % keep_count(head_keep, 8), "bf16", 64,
                    (256, 256, 256, 256), 256, 8, 2, 32, 1024,
                    keep_count(head_keep, 8), keep_count(0.5, 1024), "all", 2)


def config4() -> Workload:
    return Workload("cfg4_full_layer", "bf16", 128, (256, 256), 384, 12, 4, 32, 1536,
                    keep_count(0.6, 12), keep_count(0.4, 1536), "thirds", 3)


def config5(B: int, T: int) -> Workload:
    return Workload("cfg5_sweep_B%d_T%d" % (B, T), "bf16", B, split_even(T, 3), 256, 8, 2,
                    32, 1024, keep_count(0.5, 8), keep_count(0.5, 1024), "cycle7", 4)


CONFIG5_CELLS = [(B, T) for B in (1, 16, 256, 4096) for T in (64, 256, 1024, 4096)]


def by_name(name: str) -> Workload:
    if name.endswith(":f16"):   # the same workload with IEEE-half tensors
        w = by_name(name[:-4])
        return w.with_(dtype="f16", name=w.name + "_f16")
    if name in ("1", "cfg1"):
        return config1()
    if name in ("2", "cfg2"):
        return config2()
    if name.startswith("3") or name.startswith("cfg3"):
        ratio = {"": 0.5, "a": 0.25, "b": 0.5, "c": 0.75}[name.replace("cfg", "")[1:]]
        return config3(ratio)
    if name in ("4", "cfg4"):
        return config4()
    if name.startswith("5:") or name.startswith("cfg5:"):
        b, t = name.split(":")[1].split("x")
        return config5(int(b), int(t))
    raise KeyError(name)


def torch_dtype(w: Workload):
    return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[w.dtype]


def token_modality_ids(w: Workload) -> np.ndarray:
    return np.concatenate([np.full((n,), j, dtype=np.int32) for j, n in enumerate(w.lengths)])


def make_masks(w: Workload, rng: np.random.Generator) -> np.ndarray:
    """Per-sample modality-present bitmasks (bit j = modality j present)."""
    B, M = w.B, w.M
    full = (1 << M) - 1
    if w.mask_rule == "all":
        return np.full((B,), full, dtype=np.uint32)
    if w.mask_rule == "dropout0.3":
        out = np.zeros((B,), dtype=np.uint32)
        for b in range(B):
            m = 0
            while m == 0:  # resample the whole mask until one modality is present
                bits = rng.random(M) >= 0.3
                m = int(sum(1 << j for j in range(M) if bits[j]))
            out[b] = m
        return out
    if w.mask_rule == "thirds":
        subsets = list(range(1, full + 1))
        n = len(subsets)
        counts = [B // n + (1 if j < B % n else 0) for j in range(n)]
        return np.concatenate([np.full((cnt,), s, dtype=np.uint32)
                               for s, cnt in zip(subsets, counts)])
    if w.mask_rule == "cycle7":
        return np.array([1 + (b % full) for b in range(B)], dtype=np.uint32)
    raise ValueError(w.mask_rule)


def present_count(w: Workload, mask: int) -> int:
    """Number of tokens whose modality bit is set in `mask`."""
    return int(sum(n for j, n in enumerate(w.lengths) if (mask >> j) & 1))


def make_sample_tables(w: Workload, masks: np.ndarray, n_samples_of: Callable[[int], int],
                       rng: np.random.Generator):
    """Sampled-key tables for the sparsity score.  For every distinct count of
    present tokens T_v that occurs, one int32 table [T_v, n_s]: row i lists the
    n_s distinct key positions (indices into the present-token list, ascending)
    on which query position i is scored.  n_s = n_samples_of(T_v) comes from the
    caller.  Subsets with equal T_v share a table.  Returns (flat int32 array,
    int64 offsets indexed by mask value, -1 where the subset does not occur)."""
    S = 1 << w.M
    offsets = np.full((S,), -1, dtype=np.int64)
    chunks: List[np.ndarray] = []
    by_tv: Dict[int, int] = {}
    pos = 0
    for s in sorted(set(int(m) for m in masks)):
        tv = present_count(w, s)
        if tv not in by_tv:
            n_s = int(n_samples_of(tv))
            # a without-replacement draw of n_s out of tv for every row:
            # the n_s smallest of tv iid uniforms, as sorted positions
            keys = rng.random((tv, tv), dtype=np.float32) if tv <= 4096 else None
            if keys is not None:
                tbl = np.sort(np.argpartition(keys, n_s - 1, axis=1)[:, :n_s], axis=1) \
                    if n_s < tv else np.tile(np.arange(tv), (tv, 1))
            else:  # very long rows: per-row choice
                tbl = np.stack([np.sort(rng.choice(tv, size=n_s, replace=False))
                                for _ in range(tv)])
            by_tv[tv] = pos
            chunks.append(tbl.astype(np.int32).reshape(-1))
            pos += tv * n_s
        offsets[s] = by_tv[tv]
    flat = np.concatenate(chunks) if chunks else np.zeros((0,), dtype=np.int32)
    return flat, offsets


def entry_major_tables(w: Workload, flat: np.ndarray, offsets: np.ndarray,
                       n_samples_of: Callable[[int], int]) -> np.ndarray:
    """The same tables with every [T_v, n_s] block stored transposed ([n_s, T_v]); offsets unchanged."""
    out = flat.copy()
    done = set()
    for s, off in enumerate(offsets):
        if off < 0 or int(off) in done:
            continue
        done.add(int(off))
        tv = present_count(w, s)
        n_s = int(n_samples_of(tv))
        out[off:off + tv * n_s] = flat[off:off + tv * n_s].reshape(tv, n_s).T.reshape(-1)
    return out


@dataclass
class Inputs:
    w: Workload
    ids: np.ndarray                 # [T] int32
    masks: np.ndarray               # [B] uint32
    scores_heads: np.ndarray        # [2^M, Hq] fp32
    scores_ch: np.ndarray           # [2^M, F]  fp32
    Q: torch.Tensor                 # [B,Hq,T,d]
    K: torch.Tensor                 # [B,Hk,T,d]
    V: torch.Tensor
    X: torch.Tensor                 # [B,T,D]
    W1: torch.Tensor                # [D,F]
    W2: torch.Tensor                # [F,D]
    sample_table: np.ndarray = field(default=None)
    table_offsets: np.ndarray = field(default=None)
    subsets: np.ndarray = field(default=None)        # distinct mask values, ascending
    list_of_sample: np.ndarray = field(default=None)  # [B] index into subsets


def generate(w: Workload, n_samples_of: Callable[[int], int], device: str = "cpu",
             tensors: bool = True) -> Inputs:
    """Draw one batch.  Draw order: scores_heads, scores_ch, masks, Q, K, V, X,
    W1, W2, sample tables.  Small tables come from numpy's default_rng(seed);
    the tensors from a torch generator on `device` seeded with the same seed
    (fp32 normal draws, rounded to nearest-even bf16 for bf16 workloads)."""
    rng = np.random.default_rng(w.seed)
    S = 1 << w.M
    scores_heads = rng.standard_normal((S, w.Hq)).astype(np.float32)
    scores_ch = rng.standard_normal((S, w.F)).astype(np.float32)
    masks = make_masks(w, rng)
    ids = token_modality_ids(w)
    dt = torch_dtype(w)
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed)

    def normal(shape, std):
        if not tensors:
            return None
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            x.mul_(std)
        return x.to(dt)

    Q = normal((w.B, w.Hq, w.T, w.d), w.act_std)
    K = normal((w.B, w.Hk, w.T, w.d), w.act_std)
    V = normal((w.B, w.Hk, w.T, w.d), w.act_std)
    X = normal((w.B, w.T, w.D), w.x_std if w.x_std is not None else w.act_std)
    W1 = normal((w.D, w.F), w.w_std)
    W2 = normal((w.F, w.D), w.w_std)
    table, offsets = make_sample_tables(w, masks, n_samples_of, rng)
    subsets = np.array(sorted(set(int(m) for m in masks)), dtype=np.uint32)
    index_of = {int(s): i for i, s in enumerate(subsets)}
    list_of_sample = np.array([index_of[int(m)] for m in masks], dtype=np.int32)
    return Inputs(w, ids, masks, scores_heads, scores_ch, Q, K, V, X, W1, W2,
                  table, offsets, subsets, list_of_sample)


@dataclass
class MoeInputs:
    X: torch.Tensor                 # [N,D]
    W1: torch.Tensor                # [E,D,F]
    W2: torch.Tensor                # [E,F,D]
    kept: np.ndarray                # [E,k_c] int32, ascending per expert
    expert_ids: np.ndarray          # [N,top_k] int32, distinct per token; -1 = slot not routed
    expert_weights: np.ndarray      # [N,top_k] float32, sum to 1 per token


def generate_moe(N: int, D: int, F: int, E: int, top_k: int, k_c: int, dtype: str = "bf16", seed: int = 0,
                 skew: float = 1.0, unrouted: float = 0.0, x_std: float = 1.0, w_std: float = 0.05,
                 device: str = "cpu") -> MoeInputs:
    """One Sparse-MoE block's inputs with a routing result drawn at random (the router itself is
    outside the pruned path).  Expert popularity follows p_e ~ (e+1)^-skew, shuffled, so that the
    per-expert token counts are uneven the way trained routers' are (skew 0: uniform); each token
    gets top_k DISTINCT experts without replacement and Dirichlet(1) weights; a fraction `unrouted`
    of the slots is marked -1 (dropped by a capacity limit, or a token that is absent)."""
    rng = np.random.default_rng(seed)
    p = (np.arange(E) + 1.0) ** -skew
    p = rng.permutation(p / p.sum())
    # Gumbel top-k = sampling without replacement in proportion to p
    keys = np.log(p)[None, :] + rng.gumbel(size=(N, E))
    expert_ids = np.argsort(-keys, axis=1)[:, :top_k].astype(np.int32)
    expert_weights = rng.dirichlet(np.ones(top_k), size=N).astype(np.float32)
    if unrouted > 0.0:
        expert_ids[rng.random((N, top_k)) < unrouted] = -1
    kept = np.stack([np.sort(rng.permutation(F)[:k_c]) for _ in range(E)]).astype(np.int32)
    dt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    normal = lambda shape, std: (torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std).to(dt)
    return MoeInputs(normal((N, D), x_std), normal((E, D, F), w_std), normal((E, F, D), w_std), kept,
                     expert_ids, expert_weights)

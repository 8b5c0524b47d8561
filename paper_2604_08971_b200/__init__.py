"""Python binding of libsentry (C ABI in include/sentry.h).

Argument marshalling only: every step of the pruned-layer path (gate selection,
sparse grouped-query attention, channel-compacted FFN) runs in the CUDA kernels
of the shared library.  PyTorch is used for device memory and streams.  There is
no CPU fallback: if the library is missing or no CUDA device is present, the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsentry.so")

SENTRY_F32, SENTRY_BF16, SENTRY_F16, SENTRY_FP8_E4M3 = 0, 1, 2, 3
STATUS_BIT_TIMEOUT, STATUS_BIT_EMPTY_MASK, STATUS_BIT_BAD_INDEX = 1, 2, 4
OPT_ATTEND_KERNEL = 1
ATTEND_AUTO, ATTEND_WARP_MMA, ATTEND_TCGEN05 = 0, 1, 2
OPT_LONG_SELECT = 2
LONG_SELECT_AUTO, LONG_SELECT_QUERY_BLOCKS, LONG_SELECT_PER_GROUP = 0, 1, 2

EXPORTS = ["sentry_create", "sentry_destroy", "sentry_get_last_status", "sentry_status_string",
           "sentry_num_active_queries", "sentry_workspace_bytes", "sentry_set_workspace",
           "sentry_gate_select", "sentry_attend_fwd", "sentry_ffn_fwd", "sentry_last_launch_count",
           "sentry_profile_enable", "sentry_profile_slots", "sentry_profile_read",
           "sentry_kernel_name", "sentry_gate_select_static", "sentry_selftest_wait_expiry", "sentry_set_option",
           "sentry_ffn_packed_bytes", "sentry_ffn_prepack", "sentry_ffn_prepack_fp8", "sentry_ffn_fwd_fp8", "sentry_ffn_fwd_packed",
           "sentry_gate_eval", "sentry_gate_layer_counts", "sentry_project_qkv", "sentry_project_out",
           "sentry_gate_select_multi", "sentry_sample_table_arrange", "sentry_gate_attend_fwd", "sentry_moe_workspace_bytes", "sentry_moe_packed_bytes", "sentry_moe_prepack", "sentry_moe_ffn_fwd"]


class AttendDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("B", "T", "Hq", "Hk", "d", "k_h", "dtype", "c", "score_mode")]


class FfnDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("B", "T", "D", "F", "k_c", "n_lists", "dtype")]


class ProjDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("B", "T", "D", "Hq", "Hk", "d", "k_h", "dtype")]


class GateSet(ctypes.Structure):
    _fields_ = [("scores", ctypes.c_void_p), ("n_units", ctypes.c_int), ("k", ctypes.c_int),
                ("masks", ctypes.c_void_p), ("n_masks", ctypes.c_int), ("kept", ctypes.c_void_p),
                ("kv_groups", ctypes.c_void_p), ("heads_per_group", ctypes.c_int)]


GATE_MAX_SETS = 4


class MoeDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "D", "F", "E", "top_k", "k_c", "dtype")]


class SentryError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, status_string(code), code))
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """dlopen libsentry.so (no compute, no CUDA call) and declare the signatures."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            "%s not found: build it with `python -m paper_2604_08971_b200.build` "
            "(there is no CPU fallback)" % p)
    lib = ctypes.CDLL(p)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.sentry_create.argtypes = [ctypes.POINTER(vp), ci]
    lib.sentry_destroy.argtypes = [vp]
    lib.sentry_get_last_status.argtypes = [vp, vp]
    lib.sentry_status_string.argtypes = [ci]
    lib.sentry_status_string.restype = ctypes.c_char_p
    lib.sentry_num_active_queries.argtypes = [ci, ci]
    lib.sentry_workspace_bytes.argtypes = [ctypes.POINTER(AttendDesc), ctypes.POINTER(FfnDesc)]
    lib.sentry_workspace_bytes.restype = ctypes.c_size_t
    lib.sentry_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.sentry_gate_select.argtypes = [vp, vp, ci, ci, vp, ci, ci, vp, vp, ci, vp]
    lib.sentry_gate_select_static.argtypes = [ci, vp, ci, ci, vp, ci, ci, vp, vp, ci, vp, vp]
    lib.sentry_attend_fwd.argtypes = [vp, ctypes.POINTER(AttendDesc), vp, vp, vp, vp, vp, vp, vp,
                                      vp, ci, vp, vp, vp, vp]
    lib.sentry_ffn_fwd.argtypes = [vp, ctypes.POINTER(FfnDesc), vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sentry_last_launch_count.argtypes = [vp]
    lib.sentry_selftest_wait_expiry.argtypes = [vp, ctypes.c_longlong, vp]
    lib.sentry_set_option.argtypes = [vp, ci, ci]
    lib.sentry_gate_eval.argtypes = [vp, ci, ci, ci, vp, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sentry_gate_layer_counts.argtypes = [vp, vp, ci, ci, vp, ci, vp, vp]
    lib.sentry_project_qkv.argtypes = [vp, ctypes.POINTER(ProjDesc), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sentry_project_out.argtypes = [vp, ctypes.POINTER(ProjDesc), vp, vp, vp, vp, vp, vp, vp]
    lib.sentry_ffn_packed_bytes.argtypes = [ctypes.POINTER(FfnDesc)]
    lib.sentry_ffn_packed_bytes.restype = ctypes.c_size_t
    lib.sentry_ffn_prepack.argtypes = [vp, ctypes.POINTER(FfnDesc), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.sentry_ffn_prepack_fp8.argtypes = [vp, ctypes.POINTER(FfnDesc), vp, vp, ctypes.c_float, ctypes.c_float, vp, vp,
                                           ctypes.c_size_t, vp]
    lib.sentry_ffn_fwd_fp8.argtypes = [vp, ctypes.POINTER(FfnDesc), vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float,
                                       ctypes.c_float, ctypes.c_float, vp, vp]
    lib.sentry_ffn_fwd_packed.argtypes = [vp, ctypes.POINTER(FfnDesc), vp, vp, vp, vp, vp, vp, vp]
    lib.sentry_gate_select_multi.argtypes = [vp, ci, ctypes.POINTER(GateSet), ci, vp]
    lib.sentry_gate_attend_fwd.argtypes = [vp, ctypes.POINTER(AttendDesc), vp, ci, vp, vp, vp, vp, vp, vp, vp, ci, vp, vp, vp, vp]
    lib.sentry_sample_table_arrange.argtypes = [vp, ci, ci, vp, vp, vp, ci, vp, vp]
    lib.sentry_moe_workspace_bytes.argtypes = [ctypes.POINTER(MoeDesc)]
    lib.sentry_moe_workspace_bytes.restype = ctypes.c_size_t
    lib.sentry_moe_packed_bytes.argtypes = [ctypes.POINTER(MoeDesc)]
    lib.sentry_moe_packed_bytes.restype = ctypes.c_size_t
    lib.sentry_moe_prepack.argtypes = [vp, ctypes.POINTER(MoeDesc), vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.sentry_moe_ffn_fwd.argtypes = [vp, ctypes.POINTER(MoeDesc), vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sentry_profile_enable.argtypes = [vp, ci]
    lib.sentry_profile_slots.argtypes = []
    lib.sentry_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float),
                                        ctypes.POINTER(ci), ci]
    lib.sentry_kernel_name.argtypes = [ci]
    lib.sentry_kernel_name.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("sentry_status_string", "sentry_workspace_bytes", "sentry_kernel_name",
                        "sentry_ffn_packed_bytes", "sentry_moe_workspace_bytes", "sentry_moe_packed_bytes"):
            getattr(lib, name).restype = ci
    if path is None:
        _lib = lib
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    return _build.build(force=force, verbose=verbose)


def status_string(code: int) -> str:
    return load_library().sentry_status_string(int(code)).decode()


def num_active_queries(T_v: int, c: int = 5) -> int:
    return int(load_library().sentry_num_active_queries(int(T_v), int(c)))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("libsentry takes device tensors (got a %s tensor)" % t.device)
    if not t.is_contiguous():
        raise ValueError("libsentry takes contiguous tensors")
    return t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SENTRY_F32
    if t.dtype == torch.bfloat16:
        return SENTRY_BF16
    if t.dtype == torch.float16:
        return SENTRY_F16
    raise ValueError("unsupported dtype %s" % t.dtype)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def gate_select_static(scores: torch.Tensor, masks: torch.Tensor, k: int, kept: torch.Tensor,
                       kv_groups: Optional[torch.Tensor] = None, heads_per_group: int = 0,
                       status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """sentry_gate_select_static: the gate selection for callers that may not allocate device
    memory.  No context, no workspace; every tensor (outputs included) comes from the caller,
    and this wrapper allocates nothing either.  Returns `kept`."""
    S, n = scores.shape
    rc = load_library().sentry_gate_select_static(
        scores.device.index or 0, _ptr(scores), S, n, _ptr(masks), masks.shape[0], int(k),
        _ptr(kept), _ptr(kv_groups), int(heads_per_group), _ptr(status), _stream())
    if rc != 0:
        raise SentryError(rc, "sentry_gate_select_static")
    return kept


class Sentry:
    """One library context on one CUDA device; owns the workspace tensor."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("libsentry needs a CUDA device; there is no CPU fallback")
        self.lib = load_library()
        self.device = int(device)
        h = ctypes.c_void_p()
        rc = self.lib.sentry_create(ctypes.byref(h), self.device)
        if rc != 0:
            raise SentryError(rc, "sentry_create")
        self.h = h
        self._ws = None
        self.ensure_workspace(1 << 20)

    def close(self):
        if getattr(self, "h", None):
            self.lib.sentry_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspace ---------------------------------------------------------
    def ensure_workspace(self, nbytes: int):
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty((int(nbytes),), dtype=torch.uint8, device="cuda:%d" % self.device)
            rc = self.lib.sentry_set_workspace(self.h, self._ws.data_ptr(), self._ws.numel())
            if rc != 0:
                raise SentryError(rc, "sentry_set_workspace")

    def workspace_bytes(self, attend: Optional[AttendDesc] = None, ffn: Optional[FfnDesc] = None) -> int:
        return int(self.lib.sentry_workspace_bytes(ctypes.byref(attend) if attend else None,
                                                   ctypes.byref(ffn) if ffn else None))

    def last_status(self) -> int:
        rc = self.lib.sentry_get_last_status(self.h, _stream())
        if rc < 0:
            raise SentryError(rc, "sentry_get_last_status")
        return rc

    def selftest_wait_expiry(self, limit_cycles: int = 100000):
        """Enqueue the wait-expiry self-test (one CTA whose wait runs out after limit_cycles)."""
        rc = self.lib.sentry_selftest_wait_expiry(self.h, int(limit_cycles), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_selftest_wait_expiry")

    def set_attend_kernel(self, which: int):
        """SENTRY_OPT_ATTEND_KERNEL: ATTEND_AUTO, ATTEND_WARP_MMA or ATTEND_TCGEN05."""
        rc = self.lib.sentry_set_option(self.h, OPT_ATTEND_KERNEL, int(which))
        if rc != 0:
            raise SentryError(rc, "sentry_set_option")

    def set_option(self, option: int, value: int):
        rc = self.lib.sentry_set_option(self.h, int(option), int(value))
        if rc != 0:
            raise SentryError(rc, "sentry_set_option")

    def last_launch_count(self) -> int:
        return int(self.lib.sentry_last_launch_count(self.h))

    def profile_enable(self, on: bool):
        self.lib.sentry_profile_enable(self.h, 1 if on else 0)

    def profile_read(self) -> dict:
        """{kernel name: (total ms, launches)} since the last read (synchronises)."""
        n = int(self.lib.sentry_profile_slots())
        ms = (ctypes.c_float * n)()
        cnt = (ctypes.c_int * n)()
        rc = self.lib.sentry_profile_read(self.h, ms, cnt, n)
        if rc != 0:
            raise SentryError(rc, "sentry_profile_read")
        return {self.lib.sentry_kernel_name(i).decode(): (float(ms[i]), int(cnt[i]))
                for i in range(n) if cnt[i] > 0}

    # -- the three calls -----------------------------------------------------
    def gate_select(self, scores: torch.Tensor, masks: torch.Tensor, k: int,
                    heads_per_group: int = 0, kept: Optional[torch.Tensor] = None):
        """sentry_gate_select: scores [S,n] fp32, masks [n_masks] int32/uint32 bit patterns.
        Returns kept [n_masks,k] int32 (and the KV-group bitmaps if heads_per_group > 0)."""
        S, n = scores.shape
        n_masks = masks.shape[0]
        assert scores.dtype == torch.float32 and masks.dtype in (torch.int32, torch.uint32)
        if kept is None:
            kept = torch.empty((n_masks, k), dtype=torch.int32, device=scores.device)
        groups = torch.empty((n_masks,), dtype=torch.int32, device=scores.device) \
            if heads_per_group > 0 else None
        self.ensure_workspace(max(1 << 20, S * k * 4 + S * 4 + 1024))
        rc = self.lib.sentry_gate_select(self.h, _ptr(scores), S, n, _ptr(masks), n_masks, int(k),
                                         _ptr(kept), _ptr(groups), int(heads_per_group), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_gate_select")
        return (kept, groups) if heads_per_group > 0 else kept

    def gate_select_multi(self, sets):
        """sentry_gate_select_multi: several selections over the same mask values in one launch.
        `sets`: list of (scores [S,n] fp32, masks [n_masks], k, heads_per_group[, kept]) tuples.  Returns one
        entry per set: kept, or (kept, kv_groups) where heads_per_group > 0."""
        arr = (GateSet * len(sets))()
        outs = []
        S = sets[0][0].shape[0]
        need = 1024
        for i, item in enumerate(sets):
            scores, masks, k, hpg = item[:4]
            kept = item[4] if len(item) > 4 else None
            assert scores.shape[0] == S and scores.dtype == torch.float32
            n_masks = masks.shape[0]
            if kept is None:
                kept = torch.empty((n_masks, k), dtype=torch.int32, device=scores.device)
            groups = torch.empty((n_masks,), dtype=torch.int32, device=scores.device) if hpg > 0 else None
            arr[i] = GateSet(_ptr(scores), scores.shape[1], int(k), _ptr(masks), n_masks, _ptr(kept), _ptr(groups),
                             int(hpg))
            outs.append((kept, groups) if hpg > 0 else kept)
            need += S * k * 4 + S * 4 + 512
        self.ensure_workspace(max(1 << 20, need))
        rc = self.lib.sentry_gate_select_multi(self.h, S, arr, len(sets), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_gate_select_multi")
        return outs

    def gate_attend_fwd(self, head_scores, k_h: int, Q, K, V, token_modality_ids, masks, sample_table=None,
                        sample_offsets=None, *, c: int = 5, score_mode: int = 0, O=None, kept_heads=None,
                        active_out=None):
        """sentry_gate_attend_fwd: head selection + attention.  Returns (O [B,k_h,T,d], kept_heads [B,k_h])."""
        desc = self.attend_desc(Q, K, k_h, c, score_mode)
        B, _, T, d = Q.shape
        if O is None:
            O = torch.empty((B, k_h, T, d), dtype=Q.dtype, device=Q.device)
        if kept_heads is None:
            kept_heads = torch.empty((B, k_h), dtype=torch.int32, device=Q.device)
        S = head_scores.shape[0]
        self.ensure_workspace(max(self.workspace_bytes(attend=desc), S * k_h * 4 + S * 4 + 1024))
        n_subsets = 0 if sample_offsets is None else sample_offsets.shape[0]
        rc = self.lib.sentry_gate_attend_fwd(self.h, ctypes.byref(desc), _ptr(head_scores), S, _ptr(Q), _ptr(K), _ptr(V),
                                             _ptr(token_modality_ids), _ptr(masks), _ptr(sample_table),
                                             _ptr(sample_offsets), n_subsets, _ptr(O), _ptr(kept_heads),
                                             _ptr(active_out), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_gate_attend_fwd")
        return O, kept_heads

    def sample_table_arrange(self, token_modality_ids, sample_table, sample_offsets, c: int = 5, out=None):
        """sentry_sample_table_arrange: the tables for score_mode 2 (entry-major, bank-friendly order)."""
        if out is None:
            out = torch.empty_like(sample_table)
        rc = self.lib.sentry_sample_table_arrange(self.h, token_modality_ids.shape[0], int(c), _ptr(token_modality_ids),
                                                  _ptr(sample_table), _ptr(sample_offsets), sample_offsets.shape[0],
                                                  _ptr(out), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_sample_table_arrange")
        return out

    def attend_desc(self, Q, K, k_h: int, c: int = 5, score_mode: int = 0) -> AttendDesc:
        B, Hq, T, d = Q.shape
        return AttendDesc(B, T, Hq, K.shape[1], d, int(k_h), _dtype_code(Q), int(c), int(score_mode))

    def attend_fwd(self, Q, K, V, kept_heads, token_modality_ids, masks, sample_table=None,
                   sample_offsets=None, *, c: int = 5, score_mode: int = 0, O=None,
                   active_out=None, active_in=None, return_active: bool = False):
        """sentry_attend_fwd.  Returns O [B,k_h,T,d] (and the active lists when asked)."""
        desc = self.attend_desc(Q, K, kept_heads.shape[1], c, score_mode)
        assert K.shape == V.shape and K.dtype == Q.dtype and V.dtype == Q.dtype
        if O is None:
            O = torch.empty((desc.B, desc.k_h, desc.T, desc.d), dtype=Q.dtype, device=Q.device)
        if return_active and active_out is None:
            U_max = num_active_queries(desc.T, c)
            active_out = torch.empty((desc.B, desc.k_h, U_max), dtype=torch.int32, device=Q.device)
        self.ensure_workspace(self.workspace_bytes(attend=desc))
        n_subsets = int(sample_offsets.shape[0]) if sample_offsets is not None else 0
        rc = self.lib.sentry_attend_fwd(self.h, ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V),
                                        _ptr(kept_heads), _ptr(token_modality_ids), _ptr(masks),
                                        _ptr(sample_table), _ptr(sample_offsets), n_subsets, _ptr(O),
                                        _ptr(active_out), _ptr(active_in), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_attend_fwd")
        return (O, active_out) if return_active else O

    def ffn_desc(self, X, W1, kept_channels) -> FfnDesc:
        B, T, D = X.shape
        n_lists, k_c = kept_channels.shape
        return FfnDesc(B, T, D, W1.shape[1], k_c, n_lists, _dtype_code(X))

    def ffn_fwd(self, X, W1, W2, kept_channels, list_of_sample=None, token_modality_ids=None,
                masks=None, Y=None):
        """sentry_ffn_fwd.  Returns Y [B,T,D]."""
        if kept_channels.dim() == 1:
            kept_channels = kept_channels[None, :]
        desc = self.ffn_desc(X, W1, kept_channels)
        assert W1.dtype == X.dtype and W2.dtype == X.dtype
        if Y is None:
            Y = torch.empty_like(X)
        self.ensure_workspace(self.workspace_bytes(ffn=desc))
        rc = self.lib.sentry_ffn_fwd(self.h, ctypes.byref(desc), _ptr(X), _ptr(W1), _ptr(W2),
                                     _ptr(kept_channels), _ptr(list_of_sample),
                                     _ptr(token_modality_ids), _ptr(masks), _ptr(Y), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_ffn_fwd")
        return Y

    def ffn_prepack(self, W1, W2, kept_channels, packed=None):
        """sentry_ffn_prepack: materialise W1[:, N], W2[N, :] of every kept list once.  Returns the
        packed buffer (a uint8 tensor) for ffn_fwd_packed."""
        if kept_channels.dim() == 1:
            kept_channels = kept_channels[None, :]
        D, F = W1.shape
        n_lists, k_c = kept_channels.shape
        desc = FfnDesc(1, 1, D, F, k_c, n_lists, _dtype_code(W1))
        nbytes = int(self.lib.sentry_ffn_packed_bytes(ctypes.byref(desc)))
        if packed is None:
            packed = torch.empty((nbytes,), dtype=torch.uint8, device=W1.device)
        rc = self.lib.sentry_ffn_prepack(self.h, ctypes.byref(desc), _ptr(W1), _ptr(W2), _ptr(kept_channels),
                                         _ptr(packed), packed.numel(), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_ffn_prepack")
        return packed

    def ffn_prepack_fp8(self, W1q, W2q, scale_w1: float, scale_w2: float, kept_channels, dtype=torch.bfloat16,
                        packed=None):
        """sentry_ffn_prepack_fp8: W1q [D,F], W2q [F,D] uint8 e4m3 codes -> packed buffer of `dtype` weights."""
        if kept_channels.dim() == 1:
            kept_channels = kept_channels[None, :]
        D, F = W1q.shape
        n_lists, k_c = kept_channels.shape
        code = {torch.float32: SENTRY_F32, torch.bfloat16: SENTRY_BF16, torch.float16: SENTRY_F16}[dtype]
        desc = FfnDesc(1, 1, D, F, k_c, n_lists, code)
        nbytes = int(self.lib.sentry_ffn_packed_bytes(ctypes.byref(desc)))
        if packed is None:
            packed = torch.empty((nbytes,), dtype=torch.uint8, device=W1q.device)
        rc = self.lib.sentry_ffn_prepack_fp8(self.h, ctypes.byref(desc), _ptr(W1q), _ptr(W2q), float(scale_w1),
                                             float(scale_w2), _ptr(kept_channels), _ptr(packed), packed.numel(), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_ffn_prepack_fp8")
        return packed

    def ffn_prepack_e4m3(self, W1q, W2q, kept_channels, packed=None):
        """sentry_ffn_prepack with dtype FP8: gathers W1q[:, N], W2q[N, :] (uint8 e4m3 codes) for sentry_ffn_fwd_fp8."""
        if kept_channels.dim() == 1:
            kept_channels = kept_channels[None, :]
        D, F = W1q.shape
        n_lists, k_c = kept_channels.shape
        desc = FfnDesc(1, 1, D, F, k_c, n_lists, SENTRY_FP8_E4M3)
        nbytes = int(self.lib.sentry_ffn_packed_bytes(ctypes.byref(desc)))
        if nbytes == 0:
            raise SentryError(-4, "sentry_ffn_packed_bytes (FP8 shape)")
        if packed is None:
            packed = torch.empty((nbytes,), dtype=torch.uint8, device=W1q.device)
        rc = self.lib.sentry_ffn_prepack(self.h, ctypes.byref(desc), _ptr(W1q), _ptr(W2q), _ptr(kept_channels),
                                         _ptr(packed), packed.numel(), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_ffn_prepack (FP8)")
        return packed

    def ffn_fwd_fp8(self, Xq, packed, F: int, k_c: int, n_lists: int, scale_x: float, scale_w1: float, scale_w2: float,
                    scale_h: float, list_of_sample=None, token_modality_ids=None, masks=None, Y=None):
        """sentry_ffn_fwd_fp8: Xq [B,T,D] uint8 e4m3 codes, packed from ffn_prepack_e4m3.  Returns Y [B,T,D] bf16."""
        B, T, D = Xq.shape
        desc = FfnDesc(B, T, D, int(F), int(k_c), int(n_lists), SENTRY_FP8_E4M3)
        if Y is None:
            Y = torch.empty((B, T, D), dtype=torch.bfloat16, device=Xq.device)
        desc16 = FfnDesc(B, T, D, int(F), int(k_c), int(n_lists), SENTRY_BF16)
        self.ensure_workspace(self.workspace_bytes(ffn=desc16))
        rc = self.lib.sentry_ffn_fwd_fp8(self.h, ctypes.byref(desc), _ptr(Xq), _ptr(packed), _ptr(list_of_sample),
                                         _ptr(token_modality_ids), _ptr(masks), float(scale_x), float(scale_w1),
                                         float(scale_w2), float(scale_h), _ptr(Y), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_ffn_fwd_fp8")
        return Y

    def ffn_fwd_packed(self, X, packed, F: int, k_c: int, n_lists: int, list_of_sample=None,
                       token_modality_ids=None, masks=None, Y=None):
        """sentry_ffn_fwd_packed.  Returns Y [B,T,D]."""
        B, T, D = X.shape
        desc = FfnDesc(B, T, D, int(F), int(k_c), int(n_lists), _dtype_code(X))
        if Y is None:
            Y = torch.empty_like(X)
        self.ensure_workspace(self.workspace_bytes(ffn=desc))
        rc = self.lib.sentry_ffn_fwd_packed(self.h, ctypes.byref(desc), _ptr(X), _ptr(packed),
                                            _ptr(list_of_sample), _ptr(token_modality_ids), _ptr(masks),
                                            _ptr(Y), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_ffn_fwd_packed")
        return Y

    def gate_eval(self, layer_offsets, zeta, gamma, W1, b1, w2, b2, return_gates: bool = False):
        """sentry_gate_eval: logits (and gates) [2^M, n_units] of SentryGate's per-unit MLP (Eq. 1)."""
        n_units, hidden, M = W1.shape
        n_layers = gamma.shape[0]
        S = 1 << M
        logits = torch.empty((S, n_units), dtype=torch.float32, device=W1.device)
        gates = torch.empty_like(logits) if return_gates else None
        rc = self.lib.sentry_gate_eval(self.h, M, hidden, n_layers, _ptr(layer_offsets), n_units, _ptr(zeta),
                                       _ptr(gamma), _ptr(W1), _ptr(b1), _ptr(w2), _ptr(b2), _ptr(logits),
                                       _ptr(gates), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_gate_eval")
        return (logits, gates) if return_gates else logits

    def gate_layer_counts(self, kept, layer_offsets):
        """sentry_gate_layer_counts: kept [n_masks, k] ascending -> counts [n_masks, n_layers]."""
        n_masks, k = kept.shape
        n_layers = layer_offsets.shape[0] - 1
        counts = torch.empty((n_masks, n_layers), dtype=torch.int32, device=kept.device)
        rc = self.lib.sentry_gate_layer_counts(self.h, _ptr(kept), n_masks, k, _ptr(layer_offsets), n_layers,
                                               _ptr(counts), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_gate_layer_counts")
        return counts

    def project_qkv(self, X, WQ, WK, WV, kept_heads, token_modality_ids, masks, Hq: int, Hk: int, d: int,
                    Q=None, K=None, V=None):
        """sentry_project_qkv.  Returns Q [B,Hq,T,d], K, V [B,Hk,T,d]; fresh outputs start at zero."""
        B, T, D = X.shape
        desc = ProjDesc(B, T, D, int(Hq), int(Hk), int(d), kept_heads.shape[1], _dtype_code(X))
        if Q is None:
            Q = torch.zeros((B, Hq, T, d), dtype=X.dtype, device=X.device)
        if K is None:
            K = torch.zeros((B, Hk, T, d), dtype=X.dtype, device=X.device)
        if V is None:
            V = torch.zeros((B, Hk, T, d), dtype=X.dtype, device=X.device)
        rc = self.lib.sentry_project_qkv(self.h, ctypes.byref(desc), _ptr(X), _ptr(WQ), _ptr(WK), _ptr(WV),
                                         _ptr(kept_heads), _ptr(token_modality_ids), _ptr(masks), _ptr(Q), _ptr(K),
                                         _ptr(V), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_project_qkv")
        return Q, K, V

    def project_out(self, A, WO, kept_heads, token_modality_ids, masks, Hq: int, out=None):
        """sentry_project_out.  A [B,k_h,T,d] -> out [B,T,D]."""
        B, k_h, T, d = A.shape
        D = WO.shape[1]
        desc = ProjDesc(B, T, D, int(Hq), 1, d, k_h, _dtype_code(A))
        if out is None:
            out = torch.empty((B, T, D), dtype=A.dtype, device=A.device)
        rc = self.lib.sentry_project_out(self.h, ctypes.byref(desc), _ptr(A), _ptr(WO), _ptr(kept_heads),
                                         _ptr(token_modality_ids), _ptr(masks), _ptr(out), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_project_out")
        return out

    def moe_prepack(self, W1, W2, kept_channels, packed=None):
        """sentry_moe_prepack: W1_e[:, N_e], W2_e[N_e, :] of every expert, once.  W1 [E,D,F]; W2 [E,F,D];
        kept_channels [E,k_c].  Returns the packed buffer for moe_ffn_fwd(packed=...)."""
        E, D, F = W1.shape
        desc = MoeDesc(1, D, F, E, 1, kept_channels.shape[1], _dtype_code(W1))
        nbytes = int(self.lib.sentry_moe_packed_bytes(ctypes.byref(desc)))
        if packed is None:
            packed = torch.empty((nbytes,), dtype=torch.uint8, device=W1.device)
        rc = self.lib.sentry_moe_prepack(self.h, ctypes.byref(desc), _ptr(W1), _ptr(W2), _ptr(kept_channels),
                                         _ptr(packed), packed.numel(), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_moe_prepack")
        return packed

    def moe_ffn_fwd(self, X, expert_ids, expert_weights, W1=None, W2=None, kept_channels=None, packed=None,
                    F: Optional[int] = None, E: Optional[int] = None, k_c: Optional[int] = None, Y=None):
        """sentry_moe_ffn_fwd.  X [N,D]; expert_ids i32, expert_weights fp32 [N,top_k]; either W1 [E,D,F],
        W2 [E,F,D], kept_channels [E,k_c], or `packed` from moe_prepack with F, E, k_c.  Returns Y [N,D]."""
        N, D = X.shape
        if packed is None:
            E, _, F = W1.shape
            k_c = kept_channels.shape[1]
        desc = MoeDesc(N, D, int(F), int(E), expert_ids.shape[1], int(k_c), _dtype_code(X))
        if Y is None:
            Y = torch.empty_like(X)
        self.ensure_workspace(int(self.lib.sentry_moe_workspace_bytes(ctypes.byref(desc))))
        rc = self.lib.sentry_moe_ffn_fwd(self.h, ctypes.byref(desc), _ptr(X), _ptr(W1), _ptr(W2),
                                         _ptr(kept_channels), _ptr(packed), _ptr(expert_ids), _ptr(expert_weights),
                                         _ptr(Y), _stream())
        if rc != 0:
            raise SentryError(rc, "sentry_moe_ffn_fwd")
        return Y

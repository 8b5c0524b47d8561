"""Float64 CPU oracle for the pruned-layer path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``sentry_oracle.c`` (plain C, written from the
paper).  Only the tests, the smoke check and the benchmark's CPU-baseline /
reference arm may import this package; the CUDA library never does, and this
package never imports the CUDA library.

Inputs may be numpy arrays or torch CPU tensors of any float dtype; they are
widened to float64 exactly (bf16, fp16 and fp32 values are representable), so the
oracle sees the same numbers the GPU reads.

Besides the wrapper, numpy functions of their own for the FP8 point (Section 5):
``e4m3_decode`` (the format written out from its definition; pinned against the
library's float8 conversion on all 256 codes, tests/test_oracle_pins.py),
``dequantise_e4m3``, ``e4m3_encode`` (nearest code, ties to even, saturating;
pinned against the library's rounding on a dense sweep and on exact midpoints)
and ``ffn_fp8`` (the pruned FFN with e4m3 operands, per-tensor scales and a
requantised hidden tile; pinned against library matmuls on the decoded operands).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sentry_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over samples).  Returns the path."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + ".tmp%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-std=c99", "-shared", "-fPIC",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_threads.restype = ctypes.c_int
        lib.oracle_num_active.restype = ctypes.c_int
        lib.oracle_num_active.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.oracle_valid_tokens.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(x) -> np.ndarray:
    if hasattr(x, "detach"):  # torch tensor
        import torch
        x = x.detach().to("cpu").to(torch.float64).numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def _u32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").numpy()
    return np.ascontiguousarray(np.asarray(x).astype(np.uint32))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def threads() -> int:
    return int(_load().oracle_threads())


def num_active(T_v: int, c: int = 5) -> int:
    """U = c * ceil(ln T_v), clamped to [1, T_v] (Section 4.4)."""
    return int(_load().oracle_num_active(int(T_v), int(c)))


def gate_select(scores, masks, k: int) -> np.ndarray:
    """Top-k units of scores[mask] per mask: score descending, lower index wins
    ties, NaN last; returned ascending by index.  scores [S, n_units] fp32."""
    if hasattr(scores, "detach"):
        scores = scores.detach().to("cpu").numpy()
    sc = np.ascontiguousarray(np.asarray(scores, dtype=np.float32))
    mk = _u32(masks)
    S, n = sc.shape
    assert 1 <= k <= n and (mk < S).all()
    kept = np.empty((mk.shape[0], k), dtype=np.int32)
    _load().oracle_gate_select(_p(sc), S, n, _p(mk), mk.shape[0], int(k), _p(kept))
    return kept


def kv_groups(kept_heads, heads_per_group: int) -> np.ndarray:
    """Bitmap of referenced KV groups, floor(h / (H_q/H_k)) (Section 4.6)."""
    kh = _i32(kept_heads)
    out = np.zeros((kh.shape[0],), dtype=np.uint32)
    _load().oracle_kv_groups(_p(kh), kh.shape[0], kh.shape[1], int(heads_per_group), _p(out))
    return out


def valid_tokens(ids, mask: int) -> np.ndarray:
    ids = _i32(ids)
    out = np.empty((ids.shape[0],), dtype=np.int32)
    n = _load().oracle_valid_tokens(_p(ids), ids.shape[0], ctypes.c_uint32(int(mask)), _p(out))
    return out[:n].copy()


def attend(Q, K, V, kept_heads, ids, masks, *, c: int = 5, score_mode: int = 0,
           sample_table=None, table_offsets=None, forced_active=None,
           return_aux: bool = False):
    """SentryAttend on the kept heads.  Q [B,Hq,T,d]; K,V [B,Hk,T,d];
    kept_heads [B,k_h]; ids [T]; masks [B].  Returns O [B,k_h,T,d] float64
    (and, with return_aux, the active token lists [B,k_h,U_max] padded with -1
    and the sparsity scores [B,k_h,T], NaN on absent tokens)."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    kh, ids, mk = _i32(kept_heads), _i32(ids), _u32(masks)
    B, Hq, T, d = Q.shape
    Hk = K.shape[1]
    assert K.shape == (B, Hk, T, d) and V.shape == K.shape and Hq % Hk == 0
    k_h = kh.shape[1]
    U_max = num_active(T, c)
    tbl = offs = None
    if score_mode == 0:
        tbl = _i32(sample_table)
        offs = np.ascontiguousarray(np.asarray(table_offsets, dtype=np.int64))
    fa = None
    if forced_active is not None:
        fa = _i32(forced_active)
        assert fa.shape == (B, k_h, U_max)
    O = np.empty((B, k_h, T, d), dtype=np.float64)
    act = np.empty((B, k_h, U_max), dtype=np.int32)
    msc = np.empty((B, k_h, T), dtype=np.float64)
    _load().oracle_attend(_p(Q), _p(K), _p(V), B, T, Hq, Hk, d, int(c), _p(kh), k_h,
                          _p(ids), _p(mk), int(score_mode), _p(tbl), _p(offs),
                          U_max, _p(fa), _p(O), _p(act), _p(msc))
    if return_aux:
        return O, act, msc
    return O


def ffn(X, W1, W2, kept_channels, list_of_sample=None, ids=None, masks=None) -> np.ndarray:
    """y = gelu_erf(x W1[:, N]) W2[N, :] per row (Section 4.6).  X [B,T,D];
    W1 [D,F]; W2 [F,D]; kept_channels [n_lists,k_c]."""
    X, W1, W2 = _f64(X), _f64(W1), _f64(W2)
    kc = _i32(kept_channels)
    if kc.ndim == 1:
        kc = kc[None, :]
    B, T, D = X.shape
    F = W1.shape[1]
    assert W1.shape == (D, F) and W2.shape == (F, D)
    los = _i32(list_of_sample) if list_of_sample is not None else None
    ii = _i32(ids) if ids is not None else None
    mk = _u32(masks) if masks is not None else None
    Y = np.empty((B, T, D), dtype=np.float64)
    _load().oracle_ffn(_p(X), _p(W1), _p(W2), B, T, D, F, _p(kc), kc.shape[1],
                       _p(los), _p(ii), _p(mk), _p(Y))
    return Y


def gate_eval(layer_offsets, zeta, gamma, W1, b1, w2, b2):
    """SentryGate (Eq. 1) for every mask value: returns (z, g), both [2^M, n_units] float64.
    W1 [n_units, hidden, M]; b1, w2 [n_units, hidden]; zeta, b2 [n_units]; gamma [n_layers]."""
    lo = _i32(layer_offsets)
    zeta, gamma, W1, b1, w2, b2 = (_f64(x) for x in (zeta, gamma, W1, b1, w2, b2))
    n_units, hidden, M = W1.shape
    n_layers = gamma.shape[0]
    assert lo.shape == (n_layers + 1,) and lo[0] == 0 and lo[-1] == n_units
    z = np.empty((1 << M, n_units), dtype=np.float64)
    g = np.empty_like(z)
    _load().oracle_gate_eval(int(M), int(hidden), int(n_layers), _p(lo), int(n_units), _p(zeta), _p(gamma),
                             _p(W1), _p(b1), _p(w2), _p(b2), _p(z), _p(g))
    return z, g


def project_qkv(X, WQ, WK, WV, kept_heads, ids, masks, Hq: int, Hk: int, d: int):
    """Pruned Q/K/V projections (Section 4.6): only the column blocks of the kept heads / referenced
    KV groups, only present tokens; everything else zero.  Returns Q [B,Hq,T,d], K, V [B,Hk,T,d]."""
    X, WQ, WK, WV = (_f64(x) for x in (X, WQ, WK, WV))
    kh, ii, mk = _i32(kept_heads), _i32(ids), _u32(masks)
    B, T, D = X.shape
    assert WQ.shape == (D, Hq * d) and WK.shape == (D, Hk * d) and WV.shape == (D, Hk * d)
    Q = np.empty((B, Hq, T, d)); K = np.empty((B, Hk, T, d)); V = np.empty((B, Hk, T, d))
    _load().oracle_project_qkv(_p(X), _p(WQ), _p(WK), _p(WV), B, T, D, Hq, Hk, d, _p(kh), kh.shape[1],
                               _p(ii), _p(mk), _p(Q), _p(K), _p(V))
    return Q, K, V


def project_out(A, WO, kept_heads, ids, masks, Hq: int):
    """Pruned output projection: A [B,k_h,T,d] (kept-list order) times the kept row blocks of W_O
    [Hq d, D]; rows of absent tokens zero.  Returns [B,T,D]."""
    A, WO = _f64(A), _f64(WO)
    kh, ii, mk = _i32(kept_heads), _i32(ids), _u32(masks)
    B, k_h, T, d = A.shape
    D = WO.shape[1]
    assert WO.shape == (Hq * d, D) and kh.shape == (B, k_h)
    out = np.empty((B, T, D))
    _load().oracle_project_out(_p(A), _p(WO), B, T, D, Hq, d, _p(kh), k_h, _p(ii), _p(mk), _p(out))
    return out


def moe_ffn(X, W1, W2, kept_channels, expert_ids, expert_weights) -> np.ndarray:
    """Sparse-MoE block with expert-internal channel pruning (Section 4.6); routing given.
    X [N,D]; W1 [E,D,F]; W2 [E,F,D]; kept_channels [E,k_c]; expert_ids, expert_weights [N,top_k]."""
    X, W1, W2, wt = _f64(X), _f64(W1), _f64(W2), _f64(expert_weights)
    kc, ex = _i32(kept_channels), _i32(expert_ids)
    N, D = X.shape
    E, _, F = W1.shape
    assert W1.shape == (E, D, F) and W2.shape == (E, F, D) and kc.shape[0] == E and ex.shape == wt.shape
    assert ex.min() >= 0 and ex.max() < E
    Y = np.empty((N, D), dtype=np.float64)
    _load().oracle_moe_ffn(_p(X), _p(W1), _p(W2), N, D, F, E, _p(kc), kc.shape[1], _p(ex), _p(wt), ex.shape[1], _p(Y))
    return Y


def e4m3_decode(codes) -> np.ndarray:
    """Value of every FP8 e4m3 code (Section 5's FP8 storage point; the format is the published
    8-bit one: sign, 4 exponent bits with bias 7, 3 fraction bits, subnormals at exponent 0, no
    infinities, exponent 15 with fraction 7 is NaN, largest finite value 448).  float64, exact."""
    c = np.asarray(codes).astype(np.uint8).astype(np.int64)
    sign = np.where((c >> 7) & 1, -1.0, 1.0)
    e = (c >> 3) & 15
    m = c & 7
    val = np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2(e.astype(np.float64) - 7.0))
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


def dequantise_e4m3(codes, scale: float, dtype: str = "bf16"):
    """decode(code) * scale as the pruned FFN takes FP8-stored weights: the product in fp32 (both
    factors are exact in fp32), rounded once to the compute type by the library's conversion."""
    import torch   # only for the library's rounding to the 16-bit types
    prod = e4m3_decode(codes).astype(np.float32) * np.float32(scale)
    t = torch.from_numpy(prod)
    return t.to({"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[dtype])


def e4m3_encode(values) -> np.ndarray:
    """Nearest e4m3 code of every value (ties to even, magnitudes beyond 448 saturate to 448;
    NaN -> the NaN code), from the format's definition: below 2^-6 the spacing is 2^-9, above it
    2^(e-3) in the binade [2^e, 2^(e+1)).  uint8."""
    v = np.asarray(values, dtype=np.float64)
    a = np.minimum(np.abs(v), 448.0)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    quantum = np.exp2(e - 3.0)
    q = np.rint(a / quantum) * quantum          # numpy rounds halves to even
    q = np.minimum(q, 448.0)
    # back to (exponent, fraction) fields
    e2 = np.floor(np.log2(np.maximum(q, 2.0 ** -6)))
    sub = q < 2.0 ** -6
    frac = np.where(sub, np.rint(q / 2.0 ** -9), np.rint(q / np.exp2(e2 - 3.0)) - 8.0)
    expf = np.where(sub, 0.0, e2 + 7.0)
    code = (expf.astype(np.int64) << 3) | frac.astype(np.int64)
    code = np.where(np.signbit(v), code | 0x80, code)
    code = np.where(np.isnan(v), 0x7F, code)
    return code.astype(np.uint8)


def ffn_fp8(Xq, W1q, W2q, kept_channels, list_of_sample, ids, masks, scale_x, scale_w1, scale_w2, scale_h) -> np.ndarray:
    """The channel-compacted FFN with FP8 (e4m3) operands and per-tensor scales (Section 5's FP8
    point taken to the arithmetic): for a present row x of sample b with kept list N,
        z   = (x_q . W1_q[:, N]) * (scale_x * scale_w1)            exact products, exact sum
        h_q = e4m3( gelu(z) / scale_h )                            exact erf; nearest e4m3, saturating
        y   = (h_q . W2_q[N, :]) * (scale_h * scale_w2)
    Scale products and the requantisation argument are taken in fp32, the precision the device
    takes them in.  Xq [B,T,D], W1q [D,F], W2q [F,D] uint8 codes; returns Y [B,T,D] float64."""
    from math import sqrt
    from scipy.special import erf
    X = e4m3_decode(Xq)
    W1 = e4m3_decode(W1q)
    W2 = e4m3_decode(W2q)
    kc = _i32(kept_channels)
    los = _i32(list_of_sample) if list_of_sample is not None else np.zeros(X.shape[0], dtype=np.int32)
    B, T, D = X.shape
    a_scale = np.float32(scale_x) * np.float32(scale_w1)
    h_inv = np.float32(1.0) / np.float32(scale_h)
    y_scale = np.float32(scale_h) * np.float32(scale_w2)
    Y = np.zeros((B, T, D), dtype=np.float64)
    for b in range(B):
        N = kc[los[b]]
        present = np.ones(T, dtype=bool) if ids is None else ((int(masks[b]) >> np.asarray(ids)) & 1).astype(bool)
        xb = X[b][present]
        z = (xb @ W1[:, N]).astype(np.float32) * a_scale
        g = 0.5 * z.astype(np.float64) * (1.0 + erf(z.astype(np.float64) / sqrt(2.0)))
        hq = e4m3_decode(e4m3_encode(g.astype(np.float32) * h_inv))
        Y[b][present] = (hq @ W2[N, :]) * np.float64(y_scale)
    return Y

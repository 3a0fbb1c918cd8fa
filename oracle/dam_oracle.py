"""ctypes front end of the CPU oracle (``dam_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the
benchmark's CPU-baseline leg; the CUDA library and its Python binding never
import this module.

The C++ file holds the arithmetic of the main path (window softmax, Box-Cox
threshold, pattern counts, match, extension, masked attention).  This module
marshals numpy arrays for it, loops over (sequence, head), and states in numpy
the two side branches of the method: the other amplifications of Appendix B
(``amplify_transform`` / ``true_mask_transform``) and the multi-sample average
of Sec. 4.2.2 (``capture_average``).  ``build_masks`` / ``attention`` chain the
paper's steps in order:

  window softmax (Sec. 3, 4.2.1) -> Box-Cox + shift (Sec. 4.2.2) -> threshold
  (Sec. 4.2.3) -> pattern counts and match (Sec. 4.2.4) -> extension (Sec. 4.3)
  -> masked softmax attention (Sec. 4.3, last paragraph).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dam_oracle.cpp")
_LIB = os.path.join(_HERE, "libdam_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain -O2, OpenMP, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
               _SRC, "-o", _LIB + ".tmp"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        for name in ("oracle_window_probs", "oracle_amplify_f64", "oracle_true_mask_f64", "oracle_true_mask_f32",
                     "oracle_pattern_counts", "oracle_match", "oracle_extended_rows",
                     "oracle_attention_rows", "oracle_num_threads"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _row_view(x: np.ndarray):
    """x: float32 [n, d] view whose last axis is contiguous -> (pointer, row stride in floats)."""
    assert x.dtype == np.float32 and x.ndim == 2 and x.strides[1] == 4
    assert x.strides[0] % 4 == 0
    return _p(x), ctypes.c_int64(x.strides[0] // 4)


def window_probs(Qh: np.ndarray, Kh: np.ndarray, L: int, scale: float) -> np.ndarray:
    """Causal softmax map of the first L tokens of one (sequence, head): float64 [L, L]."""
    d = Qh.shape[1]
    P = np.empty((L, L), dtype=np.float64)
    qp, qs = _row_view(Qh)
    kp, ks = _row_view(Kh)
    rc = _load().oracle_window_probs(qp, kp, ctypes.c_int(L), ctypes.c_int(d), qs, ks,
                                     ctypes.c_double(scale), _p(P))
    assert rc == 0
    return P


def amplify_f64(P: np.ndarray, lam: float, eps: float) -> np.ndarray:
    """Box-Cox amplified, minimum-shifted map (the paper's A-tilde) of a float64 array."""
    P = np.ascontiguousarray(P, dtype=np.float64)
    out = np.empty_like(P)
    rc = _load().oracle_amplify_f64(_p(P), ctypes.c_int64(P.size), ctypes.c_double(lam),
                                    ctypes.c_double(eps), _p(out))
    assert rc == 0
    return out


def true_mask_f64(P: np.ndarray, tau: float, lam: float, eps: float) -> np.ndarray:
    P = np.ascontiguousarray(P, dtype=np.float64)
    L = P.shape[0]
    assert P.shape == (L, L)
    M = np.empty((L, L), dtype=np.uint8)
    rc = _load().oracle_true_mask_f64(_p(P), ctypes.c_int(L), ctypes.c_double(tau), ctypes.c_double(lam),
                                      ctypes.c_double(eps), _p(M))
    assert rc == 0
    return M


def true_mask_f32(P: np.ndarray, tau: float, eps: float) -> np.ndarray:
    """Threshold rule on an fp32 score tensor, evaluated in IEEE single precision (lambda = 0.5)."""
    assert P.dtype == np.float32
    P = np.ascontiguousarray(P)
    L = P.shape[0]
    assert P.shape == (L, L)
    M = np.empty((L, L), dtype=np.uint8)
    rc = _load().oracle_true_mask_f32(_p(P), ctypes.c_int(L), ctypes.c_float(tau), ctypes.c_float(eps), _p(M))
    assert rc == 0
    return M


def pattern_counts(M: np.ndarray):
    M = np.ascontiguousarray(M, dtype=np.uint8)
    L = M.shape[0]
    cntD = np.empty(L, dtype=np.int32)
    cntV = np.empty(L, dtype=np.int32)
    rc = _load().oracle_pattern_counts(_p(M), ctypes.c_int(L), _p(cntD), _p(cntV))
    assert rc == 0
    return cntD, cntV


def match(cntD: np.ndarray, cntV: np.ndarray, mu: float, min_support: int = 1):
    L = cntD.shape[0]
    D = np.empty(L, dtype=np.uint8)
    V = np.empty(L, dtype=np.uint8)
    rc = _load().oracle_match(_p(np.ascontiguousarray(cntD, dtype=np.int32)),
                              _p(np.ascontiguousarray(cntV, dtype=np.int32)),
                              ctypes.c_int(L), ctypes.c_float(mu), ctypes.c_int(min_support), _p(D), _p(V))
    assert rc == 0
    return D, V


def extended_rows(M: np.ndarray, D: np.ndarray, V: np.ndarray, S: int, rows: Sequence[int]) -> np.ndarray:
    """Rows of the S x S mask (true mask inside the window, matched patterns below it): uint8 [len(rows), S]."""
    M = np.ascontiguousarray(M, dtype=np.uint8)
    L = M.shape[0]
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    out = np.empty((rows.shape[0], S), dtype=np.uint8)
    rc = _load().oracle_extended_rows(_p(M), _p(np.ascontiguousarray(D, dtype=np.uint8)),
                                      _p(np.ascontiguousarray(V, dtype=np.uint8)),
                                      ctypes.c_int(L), ctypes.c_int(S), _p(rows), ctypes.c_int(rows.shape[0]),
                                      _p(out))
    assert rc == 0, rc
    return out


def attention_rows(Qh: np.ndarray, Kh: np.ndarray, Vh: np.ndarray, rows: Sequence[int],
                   mask_rows: Optional[np.ndarray], causal: bool, scale: float):
    """Masked softmax attention for the given query rows of one (sequence, head) over all S keys.

    Returns (O float64 [len(rows), d], LSE float64 [len(rows)])."""
    S, d = Kh.shape
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    n = rows.shape[0]
    O = np.empty((n, d), dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    qp, qs = _row_view(Qh)
    kp, ks = _row_view(Kh)
    vp, vs = _row_view(Vh)
    if mask_rows is not None:
        mask_rows = np.ascontiguousarray(mask_rows, dtype=np.uint8)
        assert mask_rows.shape == (n, S)
        mp = _p(mask_rows)
    else:
        mp = ctypes.c_void_p(0)
    rc = _load().oracle_attention_rows(qp, kp, vp, ctypes.c_int(S), ctypes.c_int(d), qs, ks, vs,
                                       ctypes.c_double(scale), _p(rows), ctypes.c_int(n), mp,
                                       ctypes.c_int(1 if causal else 0), _p(O), _p(lse))
    assert rc == 0, rc
    return O, lse


def amplify_transform(P: np.ndarray, method: str, lam: float, eps: float) -> np.ndarray:
    """Appendix B: the amplification methods on X = max(P, eps), in float64 (z-score and min-max take their
    statistics over every cell of the map), followed by the subtraction of the minimum over the whole map
    (cells above the diagonal included)."""
    X = np.maximum(np.asarray(P, dtype=np.float64), np.float64(eps))
    if method == "boxcox":
        T = np.log(X) if lam == 0 else (np.power(X, lam) - 1.0) / lam
    elif method == "log":
        T = np.log(X)
    elif method == "sqrt":
        T = np.sqrt(X)
    elif method == "arcsinh":
        T = np.log(X + np.sqrt(X * X + 1.0))
    elif method == "yeo_johnson":                       # X >= 0 branch only: X = max(P, eps) > 0
        T = np.log(X + 1.0) if lam == 0 else (np.power(X + 1.0, lam) - 1.0) / lam
    elif method in ("average", "sum"):                  # the map as it is: the average, or (method 1) the raw sum
        T = X.copy()
    elif method == "zscore":                            # statistics over every cell of the map, population deviation
        T = (X - X.mean()) / (X.std() + np.float64(eps))
    elif method == "minmax":
        T = (X - X.min()) / (X.max() - X.min() + np.float64(eps))
    else:
        raise ValueError(method)
    return T - T.min()


def true_mask_transform(P: np.ndarray, tau: float, method: str, lam: float, eps: float) -> np.ndarray:
    """Sec. 4.2.3 on an Appendix-B amplification: M = [A_tilde >= tau], nothing above the diagonal."""
    At = amplify_transform(P, method, lam, eps)
    return np.tril(At >= np.float64(tau)).astype(np.uint8)


def capture_average(samples: Sequence[np.ndarray], pcl_max: int, eps: float, dtype=np.float64):
    """Sec. 4.2.2, the averaged attention map of one head over several inputs.

    samples: window maps P_b, each [L_b, L_b] with L_b <= pcl_max (zero above the diagonal).
    A[i, j] = sum_b P_b[i, j] over the samples that contain the pair, C[i, j] = their number (a causal pair
    (i, j <= i) is contained exactly when L_b > i), A_bar = A / (C + eps).  Returns (A_bar [pcl_max, pcl_max], C
    int32 [pcl_max] per row).  With dtype float32 every sum and the division are IEEE single operations taken
    in sample order, which is the arithmetic two implementations can agree on bit for bit."""
    A = np.zeros((pcl_max, pcl_max), dtype=dtype)
    C = np.zeros(pcl_max, dtype=np.int32)
    for P in samples:
        L = P.shape[0]
        assert P.shape == (L, L) and L <= pcl_max
        A[:L, :L] = A[:L, :L] + np.tril(P).astype(dtype)
        C[:L] += 1
    den = C.astype(dtype) + dtype(eps)
    return (A / den[:, None]).astype(dtype), C


# ----------------------------------------------------------------------------------------------
# Chained helpers
# ----------------------------------------------------------------------------------------------
@dataclass
class HeadMask:
    """Mask content of one (sequence, query head): the true mask and the matched pattern sets."""
    S: int
    L: int
    M: np.ndarray      # uint8 [L, L]
    D: np.ndarray      # uint8 [L]   matched diagonal offsets
    V: np.ndarray      # uint8 [L]   matched columns
    cntD: np.ndarray
    cntV: np.ndarray
    P: Optional[np.ndarray] = None   # float64 [L, L] when kept

    def rows(self, rows: Sequence[int]) -> np.ndarray:
        return extended_rows(self.M, self.D, self.V, self.S, rows)


def head_mask_from_probs(P, S: int, tau: float, mu: float, lam: float = 0.5, eps: float = 1e-8,
                         min_support: int = 1, keep_probs: bool = False, method: str = "boxcox") -> HeadMask:
    """Steps after the attention map.  fp32 input -> the single-precision threshold chain (Box-Cox, lambda 0.5);
    any other amplification is decided in float64 with tau, eps, lambda taken at their float32 values."""
    L = P.shape[0]
    if method != "boxcox" or (P.dtype == np.float32 and lam != 0.5):
        f = np.float32
        M = true_mask_transform(P, float(f(tau)), method, float(f(lam)), float(f(eps)))
    elif P.dtype == np.float32:
        assert lam == 0.5
        M = true_mask_f32(P, tau, eps)
    else:
        M = true_mask_f64(P, tau, lam, eps)
    cntD, cntV = pattern_counts(M)
    D, V = match(cntD, cntV, mu, min_support)
    return HeadMask(S=S, L=L, M=M, D=D, V=V, cntD=cntD, cntV=cntV, P=P if keep_probs else None)


def build_masks(Q: np.ndarray, K: np.ndarray, cu_seqlens: Sequence[int], pcl_max: int, tau: float, mu: float,
                lam: float = 0.5, eps: float = 1e-8, scale: Optional[float] = None, min_support: int = 1,
                P_in: Optional[List[List[np.ndarray]]] = None, keep_probs: bool = False,
                heads: Optional[Sequence[int]] = None) -> List[List[Optional[HeadMask]]]:
    """Q float32 [T, Hq, d], K float32 [T, Hkv, d] (packed sequences) -> masks[seq][head].

    Query head h reads K of KV head h // (Hq // Hkv).  ``P_in[seq][head]`` (fp32 [L, L]) replaces the
    window softmax when both sides must start from the same score tensor."""
    T, Hq, d = Q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    if scale is None:
        scale = 1.0 / float(np.sqrt(d))
    out: List[List[Optional[HeadMask]]] = []
    for b in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        S = t1 - t0
        L = min(S, pcl_max)
        per_head: List[Optional[HeadMask]] = []
        for h in range(Hq):
            if heads is not None and h not in heads:
                per_head.append(None)
                continue
            if P_in is not None:
                P = P_in[b][h]
            else:
                P = window_probs(Q[t0:t1, h, :], K[t0:t1, h // g, :], L, scale)
            per_head.append(head_mask_from_probs(P, S, tau, mu, lam, eps, min_support, keep_probs))
        out.append(per_head)
    return out


def attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, cu_seqlens: Sequence[int], seq: int, head: int,
              rows: Sequence[int], mask: Optional[HeadMask], causal: bool = True,
              scale: Optional[float] = None, mask_rows: Optional[np.ndarray] = None):
    """O (float64 [n, d]) and LSE for query rows ``rows`` (indices within the sequence) of (seq, head)."""
    T, Hq, d = Q.shape
    g = Hq // K.shape[1]
    if scale is None:
        scale = 1.0 / float(np.sqrt(d))
    t0, t1 = int(cu_seqlens[seq]), int(cu_seqlens[seq + 1])
    if mask_rows is None and mask is not None:
        mask_rows = mask.rows(rows)
    return attention_rows(Q[t0:t1, head, :], K[t0:t1, head // g, :], V[t0:t1, head // g, :], rows, mask_rows,
                          causal, scale)

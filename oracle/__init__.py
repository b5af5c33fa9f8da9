"""CPU oracle of the MustDrop dual-attention filter: TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``mustdrop_oracle.c`` (plain C, double arithmetic, written from the
paper's Eq. 1 and Eq. 8-10) plus the numpy context functions in ``oracle.context``.  Nothing
here imports or is imported by the CUDA package; only tests, the smoke check and the
benchmark's CPU-baseline leg may use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mustdrop_oracle.c")
_LIB = os.path.join(_HERE, "libmustdrop_oracle.so")

MODE_BUDGET, MODE_THRESHOLD = 0, 1
CRIT_DUAL, CRIT_GLOBAL_ONLY, CRIT_INDIVIDUAL_ONLY = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
                               "-fno-fast-math", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("mustdrop_oracle_attention", "mustdrop_oracle_score", "mustdrop_oracle_score_per_head",
                     "mustdrop_oracle_select",
                     "mustdrop_oracle_compact"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def attention(q_text: np.ndarray, k: np.ndarray, txt_start: int, causal: bool = True,
              scale: float = 0.0) -> np.ndarray:
    """Text-row attention map of one request: q_text [H,N,D], k [H,L,D] (bf16 bits) -> p [H,N,L] float64."""
    q_text, k = _c(q_text, np.uint16), _c(k, np.uint16)
    H, N, D = q_text.shape
    L = k.shape[1]
    assert k.shape == (H, L, D)
    p = np.empty((H, N, L), np.float64)
    rc = _load().mustdrop_oracle_attention(_p(q_text), _p(k), H, N, L, D, int(txt_start), int(bool(causal)),
                                           ctypes.c_double(scale), _p(p))
    if rc:
        raise ValueError("mustdrop_oracle_attention rejected its arguments")
    return p


def score(q_text: np.ndarray, k: np.ndarray, vis_start: int, n_vis: int, txt_start: int,
          causal: bool = True, scale: float = 0.0, return_a: bool = False):
    """q_text [B,H,N,D], k [B,H,L,D] (bf16 bits) -> G, I fp32 [B,M] (and a float64 [B,N,M])."""
    q_text, k = _c(q_text, np.uint16), _c(k, np.uint16)
    B, H, N, D = q_text.shape
    L = k.shape[2]
    assert k.shape == (B, H, L, D)
    G = np.empty((B, n_vis), np.float32)
    I = np.empty((B, n_vis), np.float32)
    a = np.empty((B, N, n_vis), np.float64) if return_a else None
    rc = _load().mustdrop_oracle_score(_p(q_text), _p(k), B, H, N, L, D, int(vis_start), int(n_vis),
                                       int(txt_start), int(bool(causal)), ctypes.c_double(scale),
                                       _p(G), _p(I), _p(a))
    if rc:
        raise ValueError("mustdrop_oracle_score rejected its arguments")
    return (G, I, a) if return_a else (G, I)


def score_per_head(q_text: np.ndarray, k: np.ndarray, vis_start: int, n_vis: int, txt_start: int,
                   causal: bool = True, scale: float = 0.0):
    """The per-head reading of Eq. 10: I = head mean of the per-head maxima over text rows; G as in score()."""
    q_text, k = _c(q_text, np.uint16), _c(k, np.uint16)
    B, H, N, D = q_text.shape
    L = k.shape[2]
    assert k.shape == (B, H, L, D)
    G = np.empty((B, n_vis), np.float32)
    I = np.empty((B, n_vis), np.float32)
    rc = _load().mustdrop_oracle_score_per_head(_p(q_text), _p(k), B, H, N, L, D, int(vis_start), int(n_vis),
                                                int(txt_start), int(bool(causal)), ctypes.c_double(scale), _p(G), _p(I))
    if rc:
        raise ValueError("mustdrop_oracle_score_per_head rejected its arguments")
    return G, I


def select(G: np.ndarray, I: np.ndarray, seq_len: int, key_idx: Optional[np.ndarray] = None,
           key_cnt: Optional[np.ndarray] = None, mode: int = MODE_BUDGET, criteria: int = CRIT_DUAL,
           budget: int = 0, gamma: float = 0.0, alpha: float = 0.0
           ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """-> kept_idx int32 [B,cap] (unused slots -1), kept_cnt int32 [B], s fp32 [B,M], T fp32 [B]."""
    G, I = _c(G, np.float32), _c(I, np.float32)
    B, M = G.shape
    if key_idx is not None:
        key_idx = _c(key_idx, np.int32).reshape(B, -1)
        key_max = key_idx.shape[1]
        key_cnt = _c(key_cnt if key_cnt is not None else np.full((B,), key_max), np.int32)
    else:
        key_max = 0
    cap = budget if mode == MODE_BUDGET else M
    kept_idx = np.full((B, max(cap, 1)), -1, np.int32)[:, :cap].copy() if cap else np.zeros((B, 0), np.int32)
    kept_cnt = np.zeros((B,), np.int32)
    s = np.empty((B, M), np.float32)
    T = np.empty((B,), np.float32)
    rc = _load().mustdrop_oracle_select(_p(G), _p(I), B, M, int(seq_len), _p(key_idx), _p(key_cnt), key_max,
                                        int(mode), int(criteria), int(budget), ctypes.c_float(gamma),
                                        ctypes.c_float(alpha), _p(kept_idx), _p(kept_cnt), _p(s), _p(T))
    if rc:
        raise ValueError("mustdrop_oracle_select rejected its arguments")
    return kept_idx, kept_cnt, s, T


def compact(kept_idx: np.ndarray, kept_cnt: np.ndarray, vis_start: int, hidden: np.ndarray,
            k: np.ndarray, v: np.ndarray, fill: int = 0):
    """hidden [B,L,hid], k/v [B,H,L,D] (bf16 bits) -> hidden_out [B,cap,hid], k_out/v_out [B,H,cap,D];
    rows at and beyond kept_cnt[b] hold ``fill``."""
    kept_idx, kept_cnt = _c(kept_idx, np.int32), _c(kept_cnt, np.int32)
    hidden, k, v = _c(hidden, np.uint16), _c(k, np.uint16), _c(v, np.uint16)
    B, cap = kept_idx.shape
    _, H, L, D = k.shape
    hid = hidden.shape[2]
    ho = np.full((B, cap, hid), fill, np.uint16)
    ko = np.full((B, H, cap, D), fill, np.uint16)
    vo = np.full((B, H, cap, D), fill, np.uint16)
    rc = _load().mustdrop_oracle_compact(_p(kept_idx), _p(kept_cnt), B, cap, H, L, D, hid, int(vis_start),
                                         _p(hidden), _p(k), _p(v), _p(ho), _p(ko), _p(vo))
    if rc:
        raise ValueError("mustdrop_oracle_compact rejected its arguments")
    return ho, ko, vo

"""Upstream and downstream context of the filter, as numpy float64: TEST INFRASTRUCTURE ONLY.

The vision-encoding stage (Local Spatial Merging, Key Retaining; Sec. 3.3) produces the
tokens and the key set O that the prefill filter consumes; the decoding stage (output-aware
cache policy, Sec. 3.5) consumes the filter's kept sets.  The paper leaves their constants and
several details unstated, so every function here is a stated reading.  READING UNPINNED,
ARITHMETIC PINNED for ``local_spatial_merge``, ``key_set`` / ``upper_fence`` and
``cache_policy``: nothing the paper prints fixes the choice of similarity, weights, tau or
fence, but the arithmetic of the reading taken is checked against values worked out by hand
(windows with exactly known cosines, rank-one logits whose softmax is written with
``math.exp``, quartiles that fall on and between elements).  ``kv_cache_mb`` is pinned to the
token/MB pairs of Tables 3 and 6.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import numpy as np


def kv_cache_mb(tokens: int, layers: int = 32, hidden: int = 4096, bytes_per_el: int = 2) -> float:
    """KV-cache size of `tokens` tokens in MB (10^6 bytes): K and V, every layer (Eq. 2)."""
    return tokens * 2 * layers * hidden * bytes_per_el / 1e6


def local_spatial_merge(tokens: np.ndarray, grid: int, window: int = 2, tau: float = 0.8,
                        return_sims: bool = False):
    """Local Spatial Merging (Sec. 3.3, Eq. 5).

    tokens [grid*grid, C] in raster order.  The grid is cut into non-overlapping
    window x window squares; for each square S_w = mean over unordered pairs of the cosine
    similarity of its tokens; if S_w > tau the square is replaced by the plain average of
    its tokens, placed at the square's first raster slot.  Returns (merged tokens
    [M', C], source slot of each output token [M']), with ``return_sims`` also S_w of every
    window (raster order of windows).
    """
    x = np.asarray(tokens, np.float64)
    assert x.shape[0] == grid * grid and grid % window == 0
    keep_rows: List[np.ndarray] = []
    slots: List[int] = []
    all_sims: List[float] = []
    unit = x / np.maximum(np.linalg.norm(x, axis=1, keepdims=True), 1e-300)
    for wy in range(0, grid, window):
        for wx in range(0, grid, window):
            ids = [(wy + dy) * grid + (wx + dx) for dy in range(window) for dx in range(window)]
            sims = [float(unit[a] @ unit[b]) for ai, a in enumerate(ids) for b in ids[ai + 1:]]
            all_sims.append(float(np.mean(sims)))
            if np.mean(sims) > tau:
                keep_rows.append(x[ids].mean(axis=0))
                slots.append(ids[0])
            else:
                for t in ids:
                    keep_rows.append(x[t])
                    slots.append(t)
    order = np.argsort(np.asarray(slots), kind="stable")
    out = (np.stack(keep_rows)[order], np.asarray(slots, np.int64)[order])
    return out + (np.asarray(all_sims),) if return_sims else out


def upper_fence(a: np.ndarray) -> float:
    """The adaptive threshold mu of Eq. 7, read as Tukey's upper fence of the values a:
    Q3 + 1.5 (Q3 - Q1), the quartiles interpolated linearly between order statistics (the
    quartile of n values sits at position (n - 1) p of the sorted list)."""
    q1, q3 = np.quantile(np.asarray(a, np.float64), [0.25, 0.75])
    return float(q3 + 1.5 * (q3 - q1))


def key_set(q_cls: np.ndarray, k: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Key Retaining (Sec. 3.3, Eq. 6-7).

    q_cls [H, D], k [H, M, D]: a_cls = head mean of softmax(q_cls k^T / sqrt(D)) over the M
    patch tokens; O = {j : a_cls[j] > mu} with the adaptive threshold read as Tukey's upper
    fence mu = Q3 + 1.5 (Q3 - Q1) of a_cls.  Returns (O ascending, a_cls).
    """
    q = np.asarray(q_cls, np.float64)
    kk = np.asarray(k, np.float64)
    z = np.einsum("hd,hmd->hm", q, kk) / np.sqrt(q.shape[-1])
    z -= z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    a = p.mean(axis=0)
    mu = upper_fence(a)
    return np.nonzero(a > mu)[0].astype(np.int32), a


def cache_policy(kept_per_layer: Sequence[np.ndarray], n_layers: int, first_sparse_layer: int = 2
                 ) -> Dict[int, np.ndarray]:
    """Output-aware cache policy (Sec. 3.5).

    kept_per_layer[l] = vision tokens (original indices, ascending) that layer l's KV cache
    holds after prefill.  S_few is the set still retained at the last layer.  During decoding
    the layers with 0-based index >= first_sparse_layer ("following the second layer") keep, of
    the vision tokens, only S_few; earlier layers keep what prefill left them.
    """
    assert len(kept_per_layer) == n_layers
    s_few = np.asarray(kept_per_layer[-1])
    out = {}
    for l in range(n_layers):
        cur = np.asarray(kept_per_layer[l])
        out[l] = cur if l < first_sparse_layer else np.intersect1d(cur, s_few)
    return out

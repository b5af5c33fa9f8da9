"""Progressive filtering over several pruning layers, with a per-request number of vision
tokens: TEST INFRASTRUCTURE ONLY (plain numpy around the C oracle, one request at a time).

Sec. 3.4 applies the dual-attention filter "from the shallow layers" on, each layer working on
what the layer before it kept; after Local Spatial Merging (Sec. 3.3) requests no longer have
the same number of vision tokens.  The set still retained after the last pruning layer is the
S_few that the decoding-stage cache policy keeps (Sec. 3.5).

Layout of a request at a layer whose buffers have room for M vision tokens: rows
[0, vis_start) prefix, [vis_start, vis_start + m) its m <= M vision tokens, then its N text
tokens directly behind them; rows after vis_start + m + N are padding and are never read.

The functions here are the dense oracle applied to each request cut to its own length, so they
inherit its pins; what is new (packing, index composition) is checked by invariants only:
PARITY UNPINNED for ``filter_layer_ragged`` and ``progressive_filter``.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np

import oracle


def filter_layer_ragged(q_text: np.ndarray, k: np.ndarray, v: np.ndarray, hidden: np.ndarray, vis_start: int,
                        vis_cnt: Sequence[int], budget: int, key_idx: Optional[np.ndarray] = None,
                        key_cnt: Optional[np.ndarray] = None, orig_idx: Optional[np.ndarray] = None,
                        rebuild: bool = False, criteria: int = oracle.CRIT_DUAL, causal: bool = True
                        ) -> Dict[str, np.ndarray]:
    """One pruning layer on a ragged batch (Eq. 8-10 per request, budget mode).

    q_text [B,H,N,D], k / v [B,H,L,D], hidden [B,L,hid] as bf16 bits, L = vis_start + M + N.
    Request b holds vis_cnt[b] vision tokens; its text keys follow them.  Thresholds default
    per request (gamma = 1 / vis_cnt[b], alpha = 2 / its own sequence length).  A request with
    fewer tokens than the budget keeps them all.

    Returns G, I and the selection score s [B,M] (zero past vis_cnt[b]), kept_idx [B,budget] (-1 unused), kept_cnt [B],
    orig_out [B,budget] (orig_idx composed with kept_idx; identity when orig_idx is None) and
    the gathered tensors: the kept vision rows only, or with ``rebuild`` the whole next
    sequence [prefix ; kept vision ; text] packed the same way (zero elsewhere).
    """
    B, H, N, D = q_text.shape
    L = k.shape[2]
    M = L - vis_start - N
    hid = hidden.shape[2]
    G = np.zeros((B, M), np.float32)
    I = np.zeros((B, M), np.float32)
    S = np.zeros((B, M), np.float32)
    kept_idx = np.full((B, budget), -1, np.int32)
    kept_cnt = np.zeros((B,), np.int32)
    orig_out = np.full((B, budget), -1, np.int32)
    rows_out = vis_start + budget + N if rebuild else budget
    ho = np.zeros((B, rows_out, hid), np.uint16)
    ko = np.zeros((B, H, rows_out, D), np.uint16)
    vo = np.zeros((B, H, rows_out, D), np.uint16)
    for b in range(B):
        m = int(vis_cnt[b])
        assert 1 <= m <= M
        lb = vis_start + m + N                       # this request's own sequence length
        g, i = oracle.score(q_text[b:b + 1], k[b:b + 1, :, :lb], vis_start, m, vis_start + m, causal=causal)
        G[b, :m], I[b, :m] = g[0], i[0]
        kb = min(budget, m)
        ki = kc = None
        if key_idx is not None:
            ki, kc = key_idx[b:b + 1], key_cnt[b:b + 1]
        idx, cnt, sc, _ = oracle.select(g, i, lb, ki, kc, budget=kb, criteria=criteria)
        S[b, :m] = sc[0]
        n = int(cnt[0])
        kept_idx[b, :n], kept_cnt[b] = idx[0, :n], n
        src = orig_idx[b] if orig_idx is not None else np.arange(M, dtype=np.int32)
        orig_out[b, :n] = src[idx[0, :n]]
        rows = vis_start + idx[0, :n]
        if rebuild:                                   # [prefix ; kept vision ; text]
            rows = np.concatenate([np.arange(vis_start), rows, vis_start + m + np.arange(N)])
        ho[b, :len(rows)] = hidden[b, rows]
        ko[b, :, :len(rows)] = k[b][:, rows]
        vo[b, :, :len(rows)] = v[b][:, rows]
    return dict(G=G, I=I, s=S, kept_idx=kept_idx, kept_cnt=kept_cnt, orig_out=orig_out, hidden_out=ho, k_out=ko, v_out=vo)


def progressive_filter(layers: List[Dict[str, np.ndarray]], vis_start: int, vis_cnt0: Sequence[int],
                       budgets: Sequence[int], key_idx: Optional[np.ndarray] = None,
                       key_cnt: Optional[np.ndarray] = None) -> List[Dict[str, np.ndarray]]:
    """The filter at successive pruning layers (Sec. 3.4; S_few of Sec. 3.5 is the last orig_out).

    layers[l] holds that layer's q_text, k, v, hidden with room for M_l vision tokens, M_0 the
    input capacity and M_l = budgets[l-1] afterwards; request b enters layer l with the tokens
    layer l-1 kept (vis_cnt = the previous kept_cnt, original ids = the previous orig_out).
    The vision encoder's key set is given for the first layer only, in first-layer indices; at
    later layers the keys are the positions its members have there.
    """
    out = []
    cnt = np.asarray(vis_cnt0, np.int32)
    orig = None
    key_orig = None
    if key_idx is not None:
        key_orig = [set(key_idx[b, :key_cnt[b]].tolist()) for b in range(len(cnt))]
    for l, (t, kp) in enumerate(zip(layers, budgets)):
        ki = kc = None
        if key_orig is not None:
            B = len(cnt)
            width = key_idx.shape[1]
            ki = np.full((B, width), -1, np.int32)
            kc = np.zeros((B,), np.int32)
            for b in range(B):
                ids = np.arange(cnt[b]) if orig is None else orig[b, :cnt[b]]
                pos = [p for p, o in enumerate(ids.tolist()) if o in key_orig[b]]
                ki[b, :len(pos)], kc[b] = pos, len(pos)
        r = filter_layer_ragged(t["q_text"], t["k"], t["v"], t["hidden"], vis_start, cnt, kp, ki, kc,
                                orig_idx=orig, rebuild=True)
        r["key_idx"], r["key_cnt"] = ki, kc
        out.append(r)
        cnt, orig = r["kept_cnt"], r["orig_out"]
    return out


def cache_compact(k_cache: np.ndarray, v_cache: np.ndarray, layer_ids: np.ndarray, layer_cnt: np.ndarray,
                  s_few: np.ndarray, s_few_cnt: np.ndarray, vis_start: int, n_tail: int):
    """Decoding-stage cache of the layers that keep only S_few (Sec. 3.5).

    k_cache / v_cache [Lyr,B,H,R,D] (bf16 bits): layer y of request b holds prefix rows
    [0, vis_start), then the vision tokens layer_ids[y,b,:layer_cnt[y,b]] (original ids,
    ascending), then n_tail further rows (text).  Output [Lyr,B,H,vis_start + cap + n_tail,D]:
    prefix, the rows of the tokens in s_few[b,:s_few_cnt[b]], the tail; zero elsewhere.
    Every member of S_few must be present in every layer given.
    """
    Lyr, B, H, R, D = k_cache.shape
    cap = s_few.shape[1]
    rows_out = vis_start + cap + n_tail
    ko = np.zeros((Lyr, B, H, rows_out, D), np.uint16)
    vo = np.zeros_like(ko)
    for y in range(Lyr):
        for b in range(B):
            ids = layer_ids[y, b, :layer_cnt[y, b]].tolist()
            where = {o: p for p, o in enumerate(ids)}
            want = s_few[b, :s_few_cnt[b]].tolist()
            rows = np.asarray(list(range(vis_start)) + [vis_start + where[o] for o in want] +
                              [vis_start + len(ids) + t for t in range(n_tail)], np.int64)
            ko[y, b, :, :len(rows)] = k_cache[y, b][:, rows]
            vo[y, b, :, :len(rows)] = v_cache[y, b][:, rows]
    return ko, vo

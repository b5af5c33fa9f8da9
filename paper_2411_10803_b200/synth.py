"""Seeded synthetic inputs for the vision-token filter.

This module only *draws numbers*: it holds none of the filter's arithmetic and
imports neither the CUDA binding nor the CPU oracle, so both can be fed the very
same bytes.  Tensors are numpy arrays; bf16 values are carried as ``uint16`` bit
patterns (round-to-nearest-even from fp32).

Shapes follow the paper's workloads: the prefill sequence is the M vision tokens
followed by the N text tokens (Sec. 3.1, "Prefilling"), 576 tokens per 336x336
image, 2880 for the high-resolution model, 2048 for 8 video frames (Tables 1, 2).
Each request is drawn from its own counter-seeded stream, so one request of a
large batch can be regenerated alone.
"""
from __future__ import annotations

import dataclasses
import hashlib
from typing import Dict, Optional

import numpy as np

HEAD_DIM = 128
BASE_SEED = 20241110


@dataclasses.dataclass(frozen=True)
class Workload:
    """Sizes and structure of one synthetic workload."""

    name: str
    batch: int
    n_vis: int            # M
    n_txt: int            # N
    n_heads: int          # H
    hidden: int           # H * HEAD_DIM for every shipped workload
    n_salient: int        # planted vision keys aligned with the text queries
    key_cnt: int          # |O|, size of the vision encoder's key-token set
    budget: int           # Kp, tokens kept
    seed: int
    vis_start: int = 0    # tokens before the image (system prompt)
    frames: int = 1       # >1: keys correlated across frames (AR(1))
    ar_rho: float = 0.0
    head_dim: int = HEAD_DIM

    @property
    def txt_start(self) -> int:
        return self.vis_start + self.n_vis

    @property
    def seq_len(self) -> int:
        return self.vis_start + self.n_vis + self.n_txt

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _w(name, idx, **kw) -> Workload:
    return Workload(name=name, seed=BASE_SEED + idx, **kw)


WORKLOADS: Dict[str, Workload] = {
    # tiny reference case: one image, 24x24 grid
    "c1_tiny": _w("c1_tiny", 1, batch=1, n_vis=576, n_txt=32, n_heads=32, hidden=4096,
                  n_salient=8, key_cnt=16, budget=64),
    # LLaVA-1.5-7B shape (Table 1, 576 tokens; budgets 192/128/64)
    "c2_llava7b_b16": _w("c2_llava7b_b16", 2, batch=16, n_vis=576, n_txt=64, n_heads=32,
                         hidden=4096, n_salient=29, key_cnt=32, budget=64),
    # the same shape at batch 64: the point the throughput target is quoted on
    "c2_llava7b_b64": _w("c2_llava7b_b64", 2, batch=64, n_vis=576, n_txt=64, n_heads=32,
                         hidden=4096, n_salient=29, key_cnt=32, budget=64),
    # LLaVA-NeXT-7B shape (Table 1 / Table 6: 2880 -> 320 tokens)
    "c3_next7b": _w("c3_next7b", 3, batch=8, n_vis=2880, n_txt=64, n_heads=32, hidden=4096,
                    n_salient=144, key_cnt=64, budget=320),
    # Video-LLaVA shape (Table 2: 8 frames, 2048 tokens)
    "c4_video": _w("c4_video", 4, batch=8, n_vis=2048, n_txt=96, n_heads=32, hidden=4096,
                   n_salient=0, key_cnt=64, budget=256, frames=8, ar_rho=0.9),
    # 13B-scale stress
    "c5_13b_b64": _w("c5_13b_b64", 5, batch=64, n_vis=576, n_txt=128, n_heads=40, hidden=5120,
                     n_salient=29, key_cnt=32, budget=64),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _request_rng(w: Workload, b: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([w.seed, b])))


def make_request(w: Workload, b: int, with_values: bool = True) -> Dict[str, np.ndarray]:
    """One request's tensors.  Draw order: q_text, k, (v, hidden), salient, key set.

    q_text [H,N,D], k [H,L,D], v [H,L,D], hidden [L,hidden] as bf16 bits;
    salient_idx int32 [n_salient] and key_idx int32 [key_cnt], both vision-relative.
    ``with_values=False`` skips v/hidden (their draws are still consumed so that the
    index sets do not depend on the flag).
    """
    rng = _request_rng(w, b)
    H, N, L, D, M = w.n_heads, w.n_txt, w.seq_len, w.head_dim, w.n_vis
    q = rng.standard_normal((H, N, D), dtype=np.float32)
    if w.frames > 1 and w.ar_rho > 0.0:
        per = M // w.frames
        k = rng.standard_normal((H, L, D), dtype=np.float32)
        vis = k[:, w.vis_start:w.vis_start + w.frames * per].reshape(H, w.frames, per, D)
        c = np.float32(np.sqrt(1.0 - w.ar_rho * w.ar_rho))
        for f in range(1, w.frames):
            vis[:, f] = np.float32(w.ar_rho) * vis[:, f - 1] + c * vis[:, f]
        k[:, w.vis_start:w.vis_start + w.frames * per] = vis.reshape(H, w.frames * per, D)
    else:
        k = rng.standard_normal((H, L, D), dtype=np.float32)
    if with_values:
        v = rng.standard_normal((H, L, D), dtype=np.float32)
        hid = rng.standard_normal((L, w.hidden), dtype=np.float32)
    else:
        # advance the stream exactly as the full draw would
        rng.standard_normal((H, L, D), dtype=np.float32)
        rng.standard_normal((L, w.hidden), dtype=np.float32)
        v = hid = None
    if w.n_salient > 0:
        sal = np.sort(rng.choice(M, size=w.n_salient, replace=False)).astype(np.int32)
        noise = rng.standard_normal((H, w.n_salient, D), dtype=np.float32)
        # the mean text-query direction of each head, taken on the bf16-rounded queries
        qm = bf16_bits_to_f32(f32_to_bf16_bits(q)).mean(axis=1)                 # [H,D]
        u = qm / np.maximum(np.linalg.norm(qm, axis=1, keepdims=True), 1e-12)
        k[:, w.vis_start + sal, :] = np.float32(0.5 * np.sqrt(D)) * u[:, None, :] + noise
    else:
        sal = np.zeros((0,), dtype=np.int32)
    if w.key_cnt > 0:
        key = np.sort(rng.choice(M, size=w.key_cnt, replace=False)).astype(np.int32)
    else:
        key = np.zeros((0,), dtype=np.int32)
    out = {
        "q_text": f32_to_bf16_bits(q),
        "k": f32_to_bf16_bits(k),
        "salient_idx": sal,
        "key_idx": key,
    }
    if with_values:
        out["v"] = f32_to_bf16_bits(v)
        out["hidden"] = f32_to_bf16_bits(hid)
    return out


def make_batch(w: Workload, with_values: bool = True, requests: Optional[range] = None) -> Dict[str, np.ndarray]:
    """Stack requests: q_text [B,H,N,D], k/v [B,H,L,D], hidden [B,L,hidden] (bf16 bits),
    key_idx int32 [B,key_max] (key_max = max(key_cnt,1), unused slots -1), key_cnt int32 [B]."""
    reqs = list(requests) if requests is not None else list(range(w.batch))
    B = len(reqs)
    H, N, L, D = w.n_heads, w.n_txt, w.seq_len, w.head_dim
    out = {
        "q_text": np.empty((B, H, N, D), np.uint16),
        "k": np.empty((B, H, L, D), np.uint16),
        "key_idx": np.full((B, max(w.key_cnt, 1)), -1, np.int32),
        "key_cnt": np.full((B,), w.key_cnt, np.int32),
        "salient_idx": np.zeros((B, w.n_salient), np.int32),
    }
    if with_values:
        out["v"] = np.empty((B, H, L, D), np.uint16)
        out["hidden"] = np.empty((B, L, w.hidden), np.uint16)
    for i, b in enumerate(reqs):
        r = make_request(w, b, with_values)
        out["q_text"][i] = r["q_text"]
        out["k"][i] = r["k"]
        out["key_idx"][i, : w.key_cnt] = r["key_idx"]
        out["salient_idx"][i] = r["salient_idx"]
        if with_values:
            out["v"][i] = r["v"]
            out["hidden"][i] = r["hidden"]
    return out


def sha256_of(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


PAD_BITS = 0x7FC0   # bf16 quiet NaN: padding rows must never influence a result


def draw_vis_cnt(w: Workload, lo: float = 0.6, hi: float = 0.95, salt: int = 7) -> np.ndarray:
    """Per-request number of vision tokens left by the spatial merge: uniform in
    [lo*M, hi*M] (the paper reports 576 -> 440 on average, Table 3), at least the key set."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([w.seed, salt])))
    m = rng.integers(max(int(lo * w.n_vis), w.key_cnt, 1), max(int(hi * w.n_vis), w.key_cnt, 1) + 1, size=w.batch)
    return m.astype(np.int32)


def pack_ragged(d: Dict[str, np.ndarray], w: Workload, vis_cnt) -> Dict[str, np.ndarray]:
    """Turn a dense batch into a ragged one (data movement only): request b keeps its first
    vis_cnt[b] vision rows, its text rows move directly behind them, every later row of k, v
    and hidden is filled with NaN bits; key indices at or beyond vis_cnt[b] are dropped."""
    out = {n: a.copy() for n, a in d.items()}
    vs, M, N = w.vis_start, w.n_vis, w.n_txt
    for b in range(d["k"].shape[0]):
        m = int(vis_cnt[b])
        for name in ("k", "v"):
            if name in out:
                a = out[name][b]
                a[:, vs + m:vs + m + N] = d[name][b][:, vs + M:vs + M + N]
                a[:, vs + m + N:] = PAD_BITS
        if "hidden" in out:
            out["hidden"][b, vs + m:vs + m + N] = d["hidden"][b, vs + M:vs + M + N]
            out["hidden"][b, vs + m + N:] = PAD_BITS
        keys = [j for j in d["key_idx"][b, :d["key_cnt"][b]].tolist() if j < m]
        out["key_idx"][b] = -1
        out["key_idx"][b, :len(keys)] = keys
        out["key_cnt"][b] = len(keys)
    out["vis_cnt"] = np.asarray(vis_cnt, np.int32).copy()
    return out


def make_vit_tokens(seed: int, batch: int, grid: int, channels: int, merge_frac: float = 0.3) -> np.ndarray:
    """Vision-encoder tokens [B, grid*grid, C] as bf16 bits: i.i.d. N(0,1), except that in a
    fraction of the 2x2 windows the four tokens are one common vector plus 5 % noise (flat image
    regions, which the spatial merge is meant to collapse)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 11])))
    x = rng.standard_normal((batch, grid, grid, channels)).astype(np.float32)
    flat = rng.random((batch, grid // 2, grid // 2)) < merge_frac
    for b, wy, wx in zip(*np.nonzero(flat)):
        base = rng.standard_normal(channels).astype(np.float32)
        x[b, 2 * wy:2 * wy + 2, 2 * wx:2 * wx + 2] = base + 0.05 * x[b, 2 * wy:2 * wy + 2, 2 * wx:2 * wx + 2]
    return f32_to_bf16_bits(x.reshape(batch, grid * grid, channels))


def make_cls_attention(seed: int, batch: int, n_heads: int, head_dim: int, n_tokens: int, n_outliers: int):
    """[CLS] query [B,H,D] and patch keys [B,H,M,D] (bf16 bits): N(0,1), with n_outliers keys per
    image pulled towards the query of every head (the tokens the key set should contain)."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 13])))
    q = rng.standard_normal((batch, n_heads, head_dim)).astype(np.float32)
    k = rng.standard_normal((batch, n_heads, n_tokens, head_dim)).astype(np.float32)
    planted = np.zeros((batch, n_outliers), np.int32)
    for b in range(batch):
        idx = np.sort(rng.choice(n_tokens, n_outliers, replace=False))
        planted[b] = idx
        unit = q[b] / np.linalg.norm(q[b], axis=1, keepdims=True)
        k[b][:, idx] += 0.6 * np.sqrt(head_dim) * unit[:, None, :]
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), planted

"""Helpers of the GPU parity tests: upload, download and the comparison rules.

Rules: importance scores within 2e-3 relative (fp32 accumulation from bf16 inputs); kept
indices bit-exact, except that tokens whose oracle scores lie within 1e-3 relative of the
oracle's cut score may swap; compacted tensors byte-identical.
"""
import concurrent.futures
import functools
import os

import numpy as np
import torch

import oracle
from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import synth

SCORE_RTOL = 2e-3
SCORE_ATOL = 1e-10
TIE_RTOL = 1e-3


# Debugging overrides of the planner (the debug_* fields of the configuration) that a test's
# fixtures want in every configuration the test builds.
DEBUG = {}

VARIANT_CODES = {"two_pass": md.MUSTDROP_DEBUG_VARIANT_TWO_PASS, "fused": md.MUSTDROP_DEBUG_VARIANT_FUSED,
                 "row_split": md.MUSTDROP_DEBUG_VARIANT_ROW_SPLIT, "grid": md.MUSTDROP_DEBUG_VARIANT_GRID}


def force(monkeypatch, variant=None, cluster=None, staged=None):
    """Force a score kernel variant / a cluster size / the separate launches for the rest of the test."""
    if variant is not None:
        monkeypatch.setitem(DEBUG, "debug_score_variant", VARIANT_CODES[variant])
    if cluster:
        monkeypatch.setitem(DEBUG, "debug_cluster", int(cluster))
    if staged is not None:
        monkeypatch.setitem(DEBUG, "debug_filter_staged", 1 if staged else 0)


def cfg(w, **kw):
    """Configuration of a workload with the test's debugging overrides."""
    return md.config_for(w, **{**DEBUG, **kw})


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_scores_close(got: np.ndarray, ref: np.ndarray, what=""):
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    tol = SCORE_RTOL * np.abs(ref.astype(np.float64)) + SCORE_ATOL
    bad = err > tol
    assert not bad.any(), "%s: %d of %d outside tolerance, worst rel %.3e" % (
        what, int(bad.sum()), bad.size, float((err / np.maximum(np.abs(ref), 1e-300)).max()))


def assert_kept_matches(got_idx, got_cnt, ref_idx, ref_cnt, ref_s, key_idx=None, key_cnt=None, exact=False):
    """Per request: identical kept sets, or differences confined to the near-tie window around the
    oracle's cut.  Whatever the case, the result must be valid: ascending, in range, key set
    included, same count."""
    B = got_idx.shape[0]
    n_swapped = 0
    for b in range(B):
        c = int(got_cnt[b])
        assert c == int(ref_cnt[b]), "request %d: count %d vs oracle %d" % (b, c, int(ref_cnt[b]))
        g = got_idx[b, :c]
        r = ref_idx[b, :c]
        assert (np.diff(g) > 0).all() and (c == 0 or (g[0] >= 0 and g[-1] < ref_s.shape[1]))
        if key_idx is not None:
            kc = int(key_cnt[b])
            keys = [j for j in key_idx[b, :kc] if 0 <= j < ref_s.shape[1]]
            assert set(keys).issubset(set(g.tolist()))
        if np.array_equal(g, r):
            continue
        assert not exact, "request %d: kept indices differ from the oracle's" % b
        only_g = np.setdiff1d(g, r)
        only_r = np.setdiff1d(r, g)
        keys = set() if key_idx is None else set(key_idx[b, :int(key_cnt[b])].tolist())
        nonkey_kept = np.array([j for j in r if j not in keys], dtype=np.int64)
        cut = float(ref_s[b, nonkey_kept].min())
        for j in np.concatenate([only_g, only_r]):
            rel = abs(float(ref_s[b, j]) - cut) / abs(cut)
            assert rel < TIE_RTOL, "request %d token %d: score %.6g vs cut %.6g (rel %.2e)" % (
                b, j, ref_s[b, j], cut, rel)
        n_swapped += len(only_g)
    return n_swapped


def host_gather(kept_idx, kept_cnt, vis_start, hidden, k, v, fill_h, fill_k, fill_v):
    """numpy indexing gather with the given indices, starting from the given fill arrays."""
    ho, ko, vo = fill_h.copy(), fill_k.copy(), fill_v.copy()
    for b in range(kept_idx.shape[0]):
        c = int(kept_cnt[b])
        rows = vis_start + kept_idx[b, :c]
        ho[b, :c] = hidden[b, rows]
        ko[b, :, :c] = k[b][:, rows]
        vo[b, :, :c] = v[b][:, rows]
    return ho, ko, vo


def oracle_scores_all_requests(d, w, per_head=False):
    """The oracle's G, I for EVERY request of a batch: the plain single-threaded C routine, one call
    per request, the calls spread over the host's cores (ctypes releases the interpreter lock)."""
    fn = oracle.score_per_head if per_head else oracle.score

    def one(b):
        return fn(d["q_text"][b:b + 1], d["k"][b:b + 1], w.vis_start, w.n_vis, w.txt_start)

    with concurrent.futures.ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as pool:
        parts = list(pool.map(one, range(w.batch)))
    return np.concatenate([p[0] for p in parts]), np.concatenate([p[1] for p in parts])


@functools.lru_cache(maxsize=1)
def full_config_reference(name):
    """Inputs of a named workload and the oracle's scores for all its requests (the workload last
    asked for is kept: the tests that share it run next to each other)."""
    w = synth.WORKLOADS[name]
    d = synth.make_batch(w)
    G, I = oracle_scores_all_requests(d, w)
    return w, d, G, I

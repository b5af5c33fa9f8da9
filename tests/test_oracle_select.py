"""Pins for the oracle's selection (Eq. 9, Eq. 10, key set always kept) and compaction."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2411_10803_b200 import synth


def _scores(seed, B=1, M=12, N=4):
    rng = np.random.default_rng(seed)
    a = rng.random((B, N, M)) ** 4 / M
    return a.sum(1).astype(np.float32), a.max(1).astype(np.float32)


def _np_s(G, I, gamma, alpha, criteria=oracle.CRIT_DUAL):
    """The per-token score in IEEE single precision, one operation per step."""
    T = np.float32(np.sum(G.astype(np.float64)))
    gt = np.float32(gamma) * T
    g = G / gt
    r = I / np.float32(alpha)
    if criteria == oracle.CRIT_GLOBAL_ONLY:
        return g, gt
    if criteria == oracle.CRIT_INDIVIDUAL_ONLY:
        return r, gt
    return np.maximum(g, r), gt


@pytest.mark.parametrize("criteria", [oracle.CRIT_DUAL, oracle.CRIT_GLOBAL_ONLY, oracle.CRIT_INDIVIDUAL_ONLY])
def test_score_arithmetic_is_fp32(criteria):
    G, I = _scores(3, B=2, M=40)
    gamma, alpha = 1.0 / 40, 2.0 / 50
    _, _, s, T = oracle.select(G, I, 50, mode=oracle.MODE_BUDGET, criteria=criteria, budget=5,
                               gamma=gamma, alpha=alpha)
    for b in range(2):
        s_ref, _ = _np_s(G[b], I[b], gamma, alpha, criteria)
        assert np.array_equal(s[b], s_ref)
        assert T[b] == np.float32(np.sum(G[b].astype(np.float64)))


def test_default_thresholds():
    G, I = _scores(4, M=30)
    a = oracle.select(G, I, 37, budget=7)
    b = oracle.select(G, I, 37, budget=7, gamma=np.float32(1.0) / np.float32(30), alpha=np.float32(2.0) / np.float32(37))
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("seed", range(6))
def test_budget_against_brute_force(seed):
    """M <= 12: among all supersets of O of the right size the chosen one maximises the score
    sum, and among maximisers it is the lexicographically smallest index tuple."""
    M = 9 + seed % 4
    G, I = _scores(100 + seed, M=M)
    if seed % 2:      # force exact ties
        G[0, 2] = G[0, 5]
        I[0, 2] = I[0, 5]
        G[0, 7] = G[0, 5]
        I[0, 7] = I[0, 5]
    rng = np.random.default_rng(seed)
    key = np.sort(rng.choice(M, size=2, replace=False)).astype(np.int32)
    for budget in range(2, M + 1):
        kept, cnt, s, _ = oracle.select(G, I, M + 4, key[None, :], np.array([2], np.int32), budget=budget)
        assert cnt[0] == budget
        chosen = tuple(kept[0])
        rest = [j for j in range(M) if j not in key]
        best, best_set = None, None
        for extra in itertools.combinations(rest, budget - 2):
            cand = tuple(sorted(list(key) + list(extra)))
            val = tuple(sorted((float(s[0, j]) for j in extra), reverse=True))
            # lexicographic on the sorted score tuple == "largest under (s desc)" element by element
            keyv = (val, tuple(-j for j in cand))
            if best is None or keyv > best:
                best, best_set = keyv, cand
        assert chosen == best_set


def test_budget_invariants_and_nesting():
    B, M = 3, 200
    G, I = _scores(7, B=B, M=M, N=9)
    rng = np.random.default_rng(1)
    key = np.stack([np.sort(rng.choice(M, 10, replace=False)) for _ in range(B)]).astype(np.int32)
    cnt = np.full((B,), 10, np.int32)
    prev = None
    for budget in (10, 11, 40, 199, 200):
        kept, kc, s, _ = oracle.select(G, I, M + 9, key, cnt, budget=budget)
        assert (kc == budget).all()
        for b in range(B):
            row = kept[b]
            assert (np.diff(row) > 0).all() and row.min() >= 0 and row.max() < M
            assert set(key[b]).issubset(set(row))
            dropped = np.setdiff1d(np.arange(M), row)
            nonkey_kept = np.setdiff1d(row, key[b])
            for j in nonkey_kept:                  # pairwise: every kept non-key token beats every dropped one
                better = (s[b, j] > s[b, dropped]) | ((s[b, j] == s[b, dropped]) & (j < dropped))
                assert better.all()
            if prev is not None:
                assert set(prev[b]).issubset(set(row))
        prev = kept
    assert np.array_equal(prev[0], np.arange(M))


def test_key_set_duplicates_and_out_of_range_are_ignored():
    G, I = _scores(9, M=20)
    key = np.array([[3, 3, -1, 25, 7, 7]], np.int32)
    kept, cnt, _, _ = oracle.select(G, I, 24, key, np.array([6], np.int32), budget=2)
    assert cnt[0] == 2 and list(kept[0]) == [3, 7]
    kept, cnt, _, _ = oracle.select(G, I, 24, key, np.array([2], np.int32), budget=1)   # only the first two entries count
    assert list(kept[0]) == [3]


def test_threshold_mode_is_the_printed_rule():
    """Eq. 9 uses <=, Eq. 10 uses <; a token is dropped only if both hold and it is not in O."""
    G = np.array([[0.25, 0.125, 0.5, 0.125, 1.0]], np.float32)      # T = 2.0
    I = np.array([[0.01, 0.01, 0.01, 0.2, 0.01]], np.float32)
    gamma, alpha = 0.125, 0.2                                            # gt = 0.25
    kept, cnt, _, T = oracle.select(G, I, 10, mode=oracle.MODE_THRESHOLD, gamma=gamma, alpha=alpha)
    assert T[0] == 2.0
    # token 0: G == gt -> in D, I small -> dropped; token 1: dropped; token 2: G > gt kept;
    # token 3: in D but I == alpha (not <) -> kept; token 4 kept
    assert list(kept[0, :cnt[0]]) == [2, 3, 4]
    kept, cnt, _, _ = oracle.select(G, I, 10, np.array([[1]], np.int32), np.array([1], np.int32),
                                    mode=oracle.MODE_THRESHOLD, gamma=gamma, alpha=alpha)
    assert list(kept[0, :cnt[0]]) == [1, 2, 3, 4]
    kept, cnt, _, _ = oracle.select(G, I, 10, mode=oracle.MODE_THRESHOLD, criteria=oracle.CRIT_GLOBAL_ONLY,
                                    gamma=gamma, alpha=alpha)
    assert list(kept[0, :cnt[0]]) == [2, 4]
    kept, cnt, _, _ = oracle.select(G, I, 10, mode=oracle.MODE_THRESHOLD, criteria=oracle.CRIT_INDIVIDUAL_ONLY,
                                    gamma=gamma, alpha=alpha)
    assert list(kept[0, :cnt[0]]) == [3]


@pytest.mark.parametrize("seed", range(4))
def test_threshold_and_budget_modes_share_one_order(seed):
    """Keep-set of the printed rule == budget mode at that size whenever no score sits on the cut."""
    M = 64
    G, I = _scores(20 + seed, M=M, N=6)
    gamma, alpha = 1.2 / M, float(np.median(I)) * 1.1
    kt, ct, s, _ = oracle.select(G, I, M + 6, mode=oracle.MODE_THRESHOLD, gamma=gamma, alpha=alpha)
    assert 0 < ct[0] < M
    assert not np.any(s == 1.0)
    # the printed rule is "keep iff s >= 1" (up to strictness at equality)
    assert set(kt[0, :ct[0]]) == set(np.nonzero(s[0] >= 1.0)[0])
    kb, cb, _, _ = oracle.select(G, I, M + 6, budget=int(ct[0]), gamma=gamma, alpha=alpha)
    assert np.array_equal(kb[0], kt[0, :ct[0]])


def test_a_token_every_text_query_looks_at_is_always_selected():
    """A planted key whose logit beats every other by >= 8 for every head and query."""
    H, N, M, D = 3, 5, 40, 16
    rng = np.random.default_rng(5)
    q = rng.standard_normal((1, H, N, D)).astype(np.float32)
    k = 0.2 * rng.standard_normal((1, H, M + N, D)).astype(np.float32)
    jstar = 17
    k[0, :, jstar] = 0.0
    qb = synth.bf16_bits_to_f64(synth.f32_to_bf16_bits(q))
    # aligned with every query of the head: use the sum of unit queries, scaled up
    u = (qb[0] / np.linalg.norm(qb[0], axis=-1, keepdims=True)).sum(1)
    k[0, :, jstar] = 30.0 * u
    kb = synth.f32_to_bf16_bits(k)
    z = np.einsum("hnd,hld->hnl", qb[0], synth.bf16_bits_to_f64(kb)[0]) / np.sqrt(D)
    margin = z[:, :, jstar] - np.delete(z, jstar, axis=2).max(-1)
    if margin.min() < 8:
        pytest.skip("construction did not reach the margin")
    G, I = oracle.score(synth.f32_to_bf16_bits(q), kb, 0, M, M)
    key = np.array([[0, 1, 2]], np.int32)
    for budget in (4, 5, 20):
        kept, _, _, _ = oracle.select(G, I, M + N, key, np.array([3], np.int32), budget=budget)
        assert jstar in kept[0]
    for crit in (oracle.CRIT_GLOBAL_ONLY, oracle.CRIT_INDIVIDUAL_ONLY):
        kept, _, _, _ = oracle.select(G, I, M + N, key, np.array([3], np.int32), budget=4, criteria=crit)
        assert jstar in kept[0]


def test_compaction_identity_and_rows():
    w = synth.WORKLOADS["c1_tiny"].with_(batch=2, n_vis=12, n_txt=3, n_heads=2, hidden=256, n_salient=0,
                                         key_cnt=0, vis_start=2)
    d = synth.make_batch(w)
    M = w.n_vis
    ident = np.tile(np.arange(M, dtype=np.int32), (2, 1))
    ho, ko, vo = oracle.compact(ident, np.array([M, M], np.int32), w.vis_start, d["hidden"], d["k"], d["v"])
    assert np.array_equal(ho, d["hidden"][:, w.vis_start:w.vis_start + M])
    assert np.array_equal(ko, d["k"][:, :, w.vis_start:w.vis_start + M])
    assert np.array_equal(vo, d["v"][:, :, w.vis_start:w.vis_start + M])
    kept = np.array([[1, 4, 11, 0], [0, 2, 3, 9]], np.int32)
    cnt = np.array([3, 4], np.int32)
    ho, ko, vo = oracle.compact(kept, cnt, w.vis_start, d["hidden"], d["k"], d["v"], fill=0xABCD)
    for b in range(2):
        for r in range(4):
            if r < cnt[b]:
                src = w.vis_start + kept[b, r]
                assert np.array_equal(ho[b, r], d["hidden"][b, src])
                assert np.array_equal(ko[b, :, r], d["k"][b, :, src])
                assert np.array_equal(vo[b, :, r], d["v"][b, :, src])
            else:
                assert (ho[b, r] == 0xABCD).all() and (ko[b, :, r] == 0xABCD).all()


def test_end_to_end_small_budget_count_and_keys():
    w = synth.WORKLOADS["c1_tiny"].with_(n_vis=64, n_txt=8, n_heads=4, hidden=512, n_salient=3, key_cnt=5, budget=16)
    d = synth.make_batch(w)
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    kept, cnt, s, _ = oracle.select(G, I, w.seq_len, d["key_idx"], d["key_cnt"], budget=w.budget)
    assert cnt[0] == w.budget and set(d["key_idx"][0]).issubset(set(kept[0]))
    ho, ko, vo = oracle.compact(kept, cnt, w.vis_start, d["hidden"], d["k"], d["v"])
    assert np.array_equal(ko[0, :, 0], d["k"][0, :, kept[0, 0]])

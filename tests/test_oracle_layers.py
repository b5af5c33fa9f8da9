"""The ragged / multi-layer oracle (oracle/layers.py): what it adds to the dense oracle is
packing and index bookkeeping, checked here by closed forms, by the dense oracle on the
special case that reduces to it, and by brute-force index invariants."""
import numpy as np
import pytest

import oracle
from oracle import layers
from paper_2411_10803_b200 import synth

TINY = synth.WORKLOADS["c1_tiny"]


@pytest.fixture(scope="module", autouse=True)
def _built():
    oracle.build()


def small(**kw):
    base = dict(batch=3, n_vis=60, n_txt=5, n_heads=2, hidden=256, n_salient=2, key_cnt=3, budget=12, vis_start=2)
    base.update(kw)
    return TINY.with_(**base)


def test_full_length_requests_reduce_to_the_dense_oracle():
    w = small()
    d = synth.make_batch(w)
    r = layers.filter_layer_ragged(d["q_text"], d["k"], d["v"], d["hidden"], w.vis_start, [w.n_vis] * w.batch,
                                   w.budget, d["key_idx"], d["key_cnt"])
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    idx, cnt, _, _ = oracle.select(G, I, w.seq_len, d["key_idx"], d["key_cnt"], budget=w.budget)
    ho, ko, vo = oracle.compact(idx, cnt, w.vis_start, d["hidden"], d["k"], d["v"])
    assert np.array_equal(r["G"], G) and np.array_equal(r["I"], I)
    assert np.array_equal(r["kept_idx"], idx) and np.array_equal(r["kept_cnt"], cnt)
    assert np.array_equal(r["orig_out"], idx)
    assert np.array_equal(r["hidden_out"], ho) and np.array_equal(r["k_out"], ko) and np.array_equal(r["v_out"], vo)


def test_identical_keys_give_the_harmonic_closed_form_at_each_requests_own_length():
    # all keys equal => every visible key gets 1 / (number of visible keys): text query i of a
    # request with m vision tokens sees vis_start + m + i + 1 keys
    w = small(key_cnt=0, n_salient=0)
    d = synth.make_batch(w)
    d["k"][:] = d["k"][:, :, :1]
    vis_cnt = np.array([60, 17, 33], np.int32)
    p = synth.pack_ragged(d, w, vis_cnt)
    r = layers.filter_layer_ragged(p["q_text"], p["k"], p["v"], p["hidden"], w.vis_start, vis_cnt, w.budget)
    for b, m in enumerate(vis_cnt):
        seen = w.vis_start + m + np.arange(w.n_txt) + 1
        assert np.allclose(r["G"][b, :m], np.sum(1.0 / seen), rtol=1e-6)
        assert np.allclose(r["I"][b, :m], 1.0 / seen[0], rtol=1e-6)
        assert np.all(r["G"][b, m:] == 0) and np.all(r["I"][b, m:] == 0)
        # all scores tie: the lowest indices are kept
        assert r["kept_idx"][b, :r["kept_cnt"][b]].tolist() == list(range(min(w.budget, m)))


def test_padding_rows_and_shorter_requests():
    w = small()
    d = synth.make_batch(w)
    vis_cnt = np.array([60, 9, 41], np.int32)          # request 1 has fewer tokens than the budget
    p = synth.pack_ragged(d, w, vis_cnt)
    r = layers.filter_layer_ragged(p["q_text"], p["k"], p["v"], p["hidden"], w.vis_start, vis_cnt, w.budget,
                                   p["key_idx"], p["key_cnt"], rebuild=True)
    assert r["kept_cnt"].tolist() == [12, 9, 12]
    assert r["kept_idx"][1, :9].tolist() == list(range(9))
    # other padding bits, same result: padding is never read
    q = {n: a.copy() for n, a in p.items()}
    for b, m in enumerate(vis_cnt):
        q["k"][b][:, w.vis_start + m + w.n_txt:] = 0x3F80
    r2 = layers.filter_layer_ragged(q["q_text"], q["k"], q["v"], q["hidden"], w.vis_start, vis_cnt, w.budget,
                                    q["key_idx"], q["key_cnt"], rebuild=True)
    assert np.array_equal(r["G"], r2["G"]) and np.array_equal(r["kept_idx"], r2["kept_idx"])
    # rebuilt sequence: prefix, kept vision rows, then the request's text rows, packed
    for b, m in enumerate(vis_cnt):
        n = r["kept_cnt"][b]
        vs, N = w.vis_start, w.n_txt
        assert np.array_equal(r["hidden_out"][b, :vs], p["hidden"][b, :vs])
        assert np.array_equal(r["hidden_out"][b, vs:vs + n], p["hidden"][b, vs + r["kept_idx"][b, :n]])
        assert np.array_equal(r["hidden_out"][b, vs + n:vs + n + N], d["hidden"][b, w.txt_start:w.txt_start + N])
        assert np.array_equal(r["k_out"][b][:, vs + n:vs + n + N], d["k"][b][:, w.txt_start:w.txt_start + N])
        assert not np.any(r["k_out"][b][:, vs + n + N:])
        # a key token below vis_cnt is always kept
        keys = set(p["key_idx"][b, :p["key_cnt"][b]].tolist())
        assert keys <= set(r["kept_idx"][b, :n].tolist())


def _layer_inputs(w, caps, cnts):
    """Fresh tensors for every layer, packed for the token counts the layer will see."""
    out = []
    for l, (cap, cnt) in enumerate(zip(caps, cnts)):
        wl = w.with_(n_vis=cap, seed=w.seed + 100 * (l + 1), key_cnt=0, n_salient=min(w.n_salient, cap))
        out.append(synth.pack_ragged(synth.make_batch(wl), wl, cnt))
    return out


def test_progressive_filter_index_bookkeeping():
    w = small(batch=4, n_vis=80, budget=0)
    budgets = [40, 20, 8]
    vis_cnt0 = np.array([80, 35, 61, 52], np.int32)
    caps = [80, 40, 20]
    cnts = [vis_cnt0]
    for kp in budgets[:-1]:
        cnts.append(np.minimum(cnts[-1], kp))
    d0 = synth.make_batch(w.with_(key_cnt=3))
    key_idx, key_cnt = d0["key_idx"], d0["key_cnt"]
    key_idx = np.minimum(key_idx, 30)                    # keep every key below the shortest request
    tensors = _layer_inputs(w, caps, cnts)
    res = layers.progressive_filter(tensors, w.vis_start, vis_cnt0, budgets, key_idx, key_cnt)
    for b in range(w.batch):
        prev = np.arange(vis_cnt0[b])
        for l, r in enumerate(res):
            n = r["kept_cnt"][b]
            assert n == min(budgets[l], len(prev))
            ids = r["orig_out"][b, :n]
            assert np.all(np.diff(ids) > 0)                                   # ascending original ids
            assert np.array_equal(ids, prev[r["kept_idx"][b, :n]])            # composition, by hand
            assert set(key_idx[b, :key_cnt[b]].tolist()) <= set(ids.tolist())  # the key set survives every layer
            prev = ids
        s_few = set(res[-1]["orig_out"][b, :res[-1]["kept_cnt"][b]].tolist())
        for r in res:
            assert s_few <= set(r["orig_out"][b, :r["kept_cnt"][b]].tolist())


def test_cache_compact_by_brute_force():
    rng = np.random.default_rng(5)
    Lyr, B, H, D, vs, tail, cap = 3, 2, 2, 128, 1, 4, 6
    layer_cnt = np.array([[10, 9], [8, 9], [7, 6]], np.int32)
    layer_ids = np.full((Lyr, B, 12), -1, np.int32)
    s_few = np.full((B, cap), -1, np.int32)
    s_few_cnt = np.array([5, 6], np.int32)
    for b in range(B):
        few = np.sort(rng.choice(40, s_few_cnt[b], replace=False))
        s_few[b, :s_few_cnt[b]] = few
        for y in range(Lyr):
            rest = np.setdiff1d(np.arange(40), few)
            extra = rng.choice(rest, layer_cnt[y, b] - s_few_cnt[b], replace=False)
            layer_ids[y, b, :layer_cnt[y, b]] = np.sort(np.concatenate([few, extra]))
    R = vs + 12 + tail
    kc = rng.integers(0, 2 ** 16, (Lyr, B, H, R, D)).astype(np.uint16)
    vc = rng.integers(0, 2 ** 16, (Lyr, B, H, R, D)).astype(np.uint16)
    ko, vo = layers.cache_compact(kc, vc, layer_ids, layer_cnt, s_few, s_few_cnt, vs, tail)
    for y in range(Lyr):
        for b in range(B):
            n = s_few_cnt[b]
            assert np.array_equal(ko[y, b][:, :vs], kc[y, b][:, :vs])
            for r, o in enumerate(s_few[b, :n]):
                pos = layer_ids[y, b].tolist().index(o)
                assert np.array_equal(vo[y, b][:, vs + r], vc[y, b][:, vs + pos])
            t0 = vs + layer_cnt[y, b]
            assert np.array_equal(ko[y, b][:, vs + n:vs + n + tail], kc[y, b][:, t0:t0 + tail])
            assert not np.any(ko[y, b][:, vs + n + tail:])

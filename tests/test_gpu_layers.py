"""GPU parity of a pruning layer on a ragged batch and of a chain of pruning layers
(mustdrop_filter_layer) against the CPU oracle of oracle/layers.py."""
import numpy as np
import pytest
import torch

import oracle
from oracle import layers
from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import build as md_build
from paper_2411_10803_b200 import synth

from parity_util import assert_kept_matches, assert_scores_close, bf16_bits, cfg, force, to_dev, to_dev_bf16

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["c1_tiny"]

PATHS = ["one_launch", "three_launches", "two_pass"]


@pytest.fixture(scope="module", autouse=True)
def _built():
    md_build.build()
    assert torch.cuda.is_available()


@pytest.fixture
def path(request, monkeypatch):
    if request.param == "three_launches":
        force(monkeypatch, staged=True)
    elif request.param == "two_pass":
        force(monkeypatch, variant="two_pass")
    return request.param


def small(**kw):
    base = dict(batch=4, n_vis=300, n_txt=19, n_heads=3, hidden=384, n_salient=3, key_cnt=6, budget=48, vis_start=3)
    base.update(kw)
    return TINY.with_(**base)


def check_layer(f, w, p, ref, rebuild):
    """Compare one layer's GPU results (in Filter f) with the oracle's dict `ref`, every request; p = the inputs."""
    sel = np.arange(w.batch)
    g, i = f.g.cpu().numpy(), f.i.cpu().numpy()
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    orig = f.orig_out.cpu().numpy()
    ho, ko, vo = bf16_bits(f.hidden_out), bf16_bits(f.k_out), bf16_bits(f.v_out)
    assert_scores_close(g[sel], ref["G"], "G")
    assert_scores_close(i[sel], ref["I"], "I")
    for n, b in enumerate(sel):
        m = int(p["vis_cnt"][b])
        assert not g[b, m:].any() and not i[b, m:].any()          # absent tokens score 0
    kidx = p["key_idx"][sel] if w.key_cnt else None
    kcnt = p["key_cnt"][sel] if w.key_cnt else None
    swapped = assert_kept_matches(idx[sel], cnt[sel], ref["kept_idx"], ref["kept_cnt"], ref["s"], kidx, kcnt)
    vs, N = w.vis_start, w.n_txt
    for n, b in enumerate(sel):
        c, m = int(cnt[b]), int(p["vis_cnt"][b])
        src = p["orig_idx"][b] if "orig_idx" in p else np.arange(w.n_vis)
        assert np.array_equal(orig[b, :c], src[idx[b, :c]])        # original ids of the kept tokens
        rows = vs + idx[b, :c]
        if rebuild:
            rows = np.concatenate([np.arange(vs), rows, vs + m + np.arange(N)])
        assert np.array_equal(ho[b, :len(rows)], p["hidden"][b, rows])
        assert np.array_equal(ko[b][:, :len(rows)], p["k"][b][:, rows])
        assert np.array_equal(vo[b][:, :len(rows)], p["v"][b][:, rows])
        assert not ho[b, len(rows):].any() and not ko[b][:, len(rows):].any()   # nothing written behind the end
        if w.key_cnt:
            kc = int(p["key_cnt"][b])
            pos = [int(np.nonzero(idx[b, :c] == j)[0][0]) for j in sorted(p["key_idx"][b, :kc].tolist())]
            assert f.key_cnt_out.cpu().numpy()[b] == kc
            assert f.key_idx_out.cpu().numpy()[b, :kc].tolist() == pos
    if swapped == 0:
        assert np.array_equal(orig[sel], ref["orig_out"])
        assert np.array_equal(ho[sel], ref["hidden_out"]) and np.array_equal(ko[sel], ref["k_out"])
        assert np.array_equal(vo[sel], ref["v_out"])
    return swapped


def run_ragged_layer(w, vis_cnt, rebuild, with_orig=False):
    d = synth.make_batch(w)
    p = synth.pack_ragged(d, w, vis_cnt)
    if with_orig:
        p["orig_idx"] = (np.arange(w.n_vis, dtype=np.int32)[None, :] * 3 + 1).repeat(w.batch, 0)
    f = md.Filter(cfg(w, flags=md.MUSTDROP_FLAG_REBUILD_SEQUENCE if rebuild else 0))
    q, k, v, hid = (to_dev_bf16(p[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = (to_dev(p["key_idx"]), to_dev(p["key_cnt"])) if w.key_cnt else (None, None)
    f.filter_layer(q, k, v, hid, ki, kc, vis_cnt=to_dev(p["vis_cnt"]),
                   orig_idx=to_dev(p["orig_idx"]) if with_orig else None, want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    sel = list(range(w.batch))
    ref = layers.filter_layer_ragged(p["q_text"][sel], p["k"][sel], p["v"][sel], p["hidden"][sel], w.vis_start,
                                     p["vis_cnt"][sel], w.budget, p["key_idx"][sel] if w.key_cnt else None,
                                     p["key_cnt"][sel] if w.key_cnt else None,
                                     orig_idx=p["orig_idx"][sel] if with_orig else None, rebuild=rebuild)
    check_layer(f, w, p, ref, rebuild)
    launches = f.filter_launches
    f.close()
    return launches


@pytest.mark.parametrize("path", PATHS, indirect=True)
@pytest.mark.parametrize("rebuild", [False, True])
def test_ragged_layer_matches_oracle(path, rebuild):
    w = small()
    launches = run_ragged_layer(w, np.array([300, 48, 131, 17], np.int32), rebuild, with_orig=rebuild)
    assert launches == {"one_launch": 1, "three_launches": 3, "two_pass": 4}[path]


@pytest.mark.parametrize("path", PATHS, indirect=True)
def test_ragged_layer_without_key_set_many_text_rows(path):
    w = small(batch=3, n_vis=200, n_txt=100, n_heads=2, hidden=256, key_cnt=0, budget=30, vis_start=0)
    run_ragged_layer(w, np.array([200, 30, 97], np.int32), True)


@pytest.mark.parametrize("cluster", [2, 3, 5])
def test_ragged_layer_with_logits_that_grow_along_the_keys(monkeypatch, cluster):
    """The careful path of the exp warps (a chunk's sum leaves its range: new stabiliser, stored
    chunks rescaled) in a ragged batch: lanes of the same warp see nothing at all of their half of
    the CTA's keys (short requests), and the rows behind a request's sequence hold NaN bits."""
    force(monkeypatch, variant="fused", cluster=cluster)
    w = small(batch=4, n_vis=600, n_txt=40, n_heads=2, hidden=256, n_salient=0, key_cnt=0, budget=64, vis_start=0)
    d = synth.make_batch(w)
    q = synth.bf16_bits_to_f32(d["q_text"])
    k = synth.bf16_bits_to_f32(d["k"])
    u = q.mean(axis=2, keepdims=True)
    u /= np.linalg.norm(u, axis=-1, keepdims=True)
    ramp = np.linspace(0.0, 160.0, w.n_vis, dtype=np.float32)[None, None, :, None]     # over the vision keys only
    k[:, :, :w.n_vis] += ramp * u * np.sqrt(128.0) / np.maximum(np.linalg.norm(q, axis=-1).mean(), 1e-6) * 3.0
    d["k"] = synth.f32_to_bf16_bits(k.astype(np.float32))
    vis_cnt = np.array([600, 150, 290, 40], np.int32)
    p = synth.pack_ragged(d, w, vis_cnt)
    f = md.Filter(cfg(w, flags=md.MUSTDROP_FLAG_REBUILD_SEQUENCE))
    qd, kd, vd, hd = (to_dev_bf16(p[n]) for n in ("q_text", "k", "v", "hidden"))
    f.filter_layer(qd, kd, vd, hd, None, None, vis_cnt=to_dev(p["vis_cnt"]), want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    assert f.score_variant == "fused_cluster_tcgen05"
    ref = layers.filter_layer_ragged(p["q_text"], p["k"], p["v"], p["hidden"], w.vis_start, p["vis_cnt"], w.budget,
                                     None, None, rebuild=True)
    g, i = f.g.cpu().numpy(), f.i.cpu().numpy()
    assert np.isfinite(g).all() and np.isfinite(i).all()
    big = ref["G"] > 1e-9                                   # compare where the mass is; the rest underflows alike
    assert big.sum() > 20
    assert_scores_close(g[big], ref["G"][big], "G")
    assert_scores_close(i[big], ref["I"][big], "I")
    assert (g[~big] <= 1e-7).all()
    for b in range(w.batch):
        assert not g[b, vis_cnt[b]:].any() and not i[b, vis_cnt[b]:].any()
    f.close()


def test_ragged_layer_llava7b_batch16():
    w = synth.WORKLOADS["c2_llava7b_b16"]
    assert run_ragged_layer(w, synth.draw_vis_cnt(w), True) == 1


def test_ragged_layer_long_sequence_falls_back_to_the_two_pass_score():
    w = synth.WORKLOADS["c4_video"].with_(batch=2, n_vis=4000, n_txt=100, n_heads=2, hidden=256, budget=300)
    assert run_ragged_layer(w, synth.draw_vis_cnt(w), True) == 4


def test_ragged_layer_video_on_a_large_cluster(monkeypatch):
    force(monkeypatch, variant="fused")
    w = synth.WORKLOADS["c4_video"].with_(batch=2)
    assert run_ragged_layer(w, synth.draw_vis_cnt(w), True) == 1


def test_ragged_layer_next7b_on_a_large_cluster(monkeypatch):
    force(monkeypatch, variant="fused")
    w = synth.WORKLOADS["c3_next7b"].with_(batch=2)
    assert run_ragged_layer(w, synth.draw_vis_cnt(w), True) == 1


@pytest.mark.parametrize("path", ["one_launch", "two_pass"], indirect=True)
def test_chain_of_three_layers_matches_oracle(path):
    w = small(batch=4, n_vis=320, key_cnt=5, n_txt=16, budget=0)
    budgets, caps = [128, 64, 24], [320, 128, 64]
    vis_cnt0 = np.array([320, 100, 251, 77], np.int32)
    cnts = [vis_cnt0]
    for kp in budgets[:-1]:
        cnts.append(np.minimum(cnts[-1], kp))
    d0 = synth.make_batch(w.with_(key_cnt=5))
    key_idx, key_cnt = np.minimum(d0["key_idx"], 70), d0["key_cnt"].copy()
    for b in range(w.batch):                      # distinct keys below the shortest request
        ks = sorted(set(key_idx[b].tolist()))
        key_idx[b] = -1
        key_idx[b, :len(ks)], key_cnt[b] = ks, len(ks)
    tensors = []
    for l, (cap, cnt) in enumerate(zip(caps, cnts)):
        wl = w.with_(n_vis=cap, seed=w.seed + 100 * (l + 1), key_cnt=0, n_salient=3)
        tensors.append(synth.pack_ragged(synth.make_batch(wl), wl, cnt))
    ref = layers.progressive_filter(tensors, w.vis_start, vis_cnt0, budgets, key_idx, key_cnt)

    # the GPU chain: every layer's outputs feed the next, no host synchronisation in between
    filters, dev = [], []
    for l, (cap, kp) in enumerate(zip(caps, budgets)):
        wl = w.with_(n_vis=cap, budget=kp)
        filters.append(md.Filter(cfg(wl, key_max=5, flags=md.MUSTDROP_FLAG_REBUILD_SEQUENCE)))
        dev.append([to_dev_bf16(tensors[l][n]) for n in ("q_text", "k", "v", "hidden")])
    ki, kc, vc, orig = to_dev(key_idx), to_dev(key_cnt), to_dev(vis_cnt0), None
    for l, f in enumerate(filters):
        q, k, v, hid = dev[l]
        f.filter_layer(q, k, v, hid, ki, kc, vis_cnt=vc, orig_idx=orig)
        ki, kc, vc, orig = f.key_idx_out, f.key_cnt_out, f.kept_cnt, f.orig_out
    torch.cuda.synchronize()
    for l, f in enumerate(filters):
        assert f.device_status() == (0, 0)
        r = ref[l]
        idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
        assert_scores_close(f.g.cpu().numpy(), r["G"], "G layer %d" % l)
        swapped = assert_kept_matches(idx, cnt, r["kept_idx"], r["kept_cnt"], r["s"], r["key_idx"], r["key_cnt"])
        assert swapped == 0, "a near-tie at layer %d: later layers cannot be compared" % l
        assert np.array_equal(f.orig_out.cpu().numpy(), r["orig_out"])
        assert np.array_equal(bf16_bits(f.hidden_out), r["hidden_out"])
        assert np.array_equal(bf16_bits(f.k_out), r["k_out"]) and np.array_equal(bf16_bits(f.v_out), r["v_out"])
        if l + 1 < len(filters):
            nk = ref[l + 1]["key_cnt"]
            assert np.array_equal(f.key_cnt_out.cpu().numpy(), nk)
            for b in range(w.batch):
                assert np.array_equal(f.key_idx_out.cpu().numpy()[b, :nk[b]], ref[l + 1]["key_idx"][b, :nk[b]])
    # S_few: what the last layer kept, in original ids, is inside every earlier layer's set
    s_few = filters[-1].orig_out.cpu().numpy()
    for b in range(w.batch):
        last = set(s_few[b, :filters[-1].kept_cnt.cpu().numpy()[b]].tolist())
        for f in filters:
            assert last <= set(f.orig_out.cpu().numpy()[b].tolist())
    for f in filters:
        f.close()


# ---- decoding-stage cache compaction -----------------------------------------------------------

def _cache_case(seed, Lyr, B, H, vs, tail, ids_max, cap, universe):
    rng = np.random.default_rng(seed)
    s_few = np.full((B, cap), -1, np.int32)
    s_few_cnt = rng.integers(1, cap + 1, B).astype(np.int32)
    layer_ids = np.full((Lyr, B, ids_max), -1, np.int32)
    layer_cnt = np.zeros((Lyr, B), np.int32)
    for b in range(B):
        few = np.sort(rng.choice(universe, s_few_cnt[b], replace=False))
        s_few[b, :s_few_cnt[b]] = few
        rest = np.setdiff1d(np.arange(universe), few)
        for y in range(Lyr):
            n = int(rng.integers(s_few_cnt[b], ids_max + 1))
            extra = rng.choice(rest, n - s_few_cnt[b], replace=False)
            layer_ids[y, b, :n] = np.sort(np.concatenate([few, extra]))
            layer_cnt[y, b] = n
    R = vs + ids_max + tail
    kc = rng.integers(0, 2 ** 16, (Lyr, B, H, R, 128)).astype(np.uint16)
    vc = rng.integers(0, 2 ** 16, (Lyr, B, H, R, 128)).astype(np.uint16)
    return kc, vc, layer_ids, layer_cnt, s_few, s_few_cnt, R


@pytest.mark.parametrize("shape", [(3, 2, 2, 1, 4, 12, 6, 40), (5, 3, 8, 0, 7, 64, 45, 576), (2, 4, 3, 5, 0, 33, 33, 100)])
def test_cache_compact_matches_oracle(shape):
    Lyr, B, H, vs, tail, ids_max, cap, universe = shape
    kc, vc, layer_ids, layer_cnt, s_few, s_few_cnt, R = _cache_case(11, *shape)
    rk, rv = layers.cache_compact(kc, vc, layer_ids, layer_cnt, s_few, s_few_cnt, vs, tail)
    rows_out = vs + cap + tail
    ko = torch.zeros((Lyr, B, H, rows_out, 128), dtype=torch.bfloat16, device="cuda")
    vo = torch.zeros_like(ko)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    st = md.mustdrop_cache_compact(to_dev_bf16(kc), to_dev_bf16(vc), to_dev(layer_ids), to_dev(layer_cnt), to_dev(s_few),
                                   to_dev(s_few_cnt), ko, vo, ws, n_layers=Lyr, batch=B, n_heads=H, rows_in=R,
                                   vis_start=vs, n_tail=tail, ids_max=ids_max, cap=cap)
    assert st == md.MUSTDROP_OK
    torch.cuda.synchronize()
    assert ws[:8].cpu().numpy().view(np.int32).tolist() == [0, 0]
    assert np.array_equal(bf16_bits(ko), rk) and np.array_equal(bf16_bits(vo), rv)


def test_cache_compact_reports_a_token_the_layer_does_not_hold_and_takes_one_tensor():
    shape = (2, 2, 2, 1, 3, 10, 5, 30)
    Lyr, B, H, vs, tail, ids_max, cap, universe = shape
    kc, vc, layer_ids, layer_cnt, s_few, s_few_cnt, R = _cache_case(3, *shape)
    gone = s_few[1, 0]
    pos = layer_ids[1, 1].tolist().index(gone)
    layer_ids[1, 1, pos] = gone - 1 if pos == 0 or layer_ids[1, 1, pos - 1] < gone - 1 else gone   # keep ascending
    missing = layer_ids[1, 1, pos] != gone
    ko = torch.zeros((Lyr, B, H, vs + cap + tail, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    st = md.mustdrop_cache_compact(to_dev_bf16(kc), None, to_dev(layer_ids), to_dev(layer_cnt), to_dev(s_few),
                                   to_dev(s_few_cnt), ko, None, ws, n_layers=Lyr, batch=B, n_heads=H, rows_in=R,
                                   vis_start=vs, n_tail=tail, ids_max=ids_max, cap=cap)
    assert st == md.MUSTDROP_OK
    torch.cuda.synchronize()
    code, detail = ws[:8].cpu().numpy().view(np.int32).tolist()
    if missing:
        assert code == md.MUSTDROP_ERR_BAD_KEY_INDEX and detail == 1 * 65536 + 0
        assert not bf16_bits(ko)[1, 1][:, vs + 0].any()                 # the row was skipped
    # every other row is the brute-force gather
    out = bf16_bits(ko)
    for y in range(Lyr):
        for b in range(B):
            ids = layer_ids[y, b, :layer_cnt[y, b]].tolist()
            for r, o in enumerate(s_few[b, :s_few_cnt[b]].tolist()):
                if o in ids:
                    assert np.array_equal(out[y, b][:, vs + r], kc[y, b][:, vs + ids.index(o)])


def test_ragged_layer_with_text_rows_in_two_launches(monkeypatch):
    force(monkeypatch, variant="row_split")
    w = small(batch=3, n_vis=260, n_txt=90, n_heads=2, hidden=256, key_cnt=4, budget=40, vis_start=2)
    assert run_ragged_layer(w, np.array([260, 40, 133], np.int32), True) == 2


@pytest.mark.parametrize("path", ["one_launch", "two_pass"], indirect=True)
def test_ragged_layer_threshold_mode_is_the_printed_rule_on_each_requests_own_sizes(path):
    # Eq. 9 and Eq. 10 as printed, with gamma = 1 / (own tokens) and alpha = 2 / (own length)
    w = small(batch=4, n_vis=280, n_txt=17, key_cnt=5)
    d = synth.make_batch(w)
    vis_cnt = np.array([280, 31, 150, 199], np.int32)
    p = synth.pack_ragged(d, w, vis_cnt)
    f = md.Filter(cfg(w, mode=md.MUSTDROP_MODE_THRESHOLD, flags=md.MUSTDROP_FLAG_REBUILD_SEQUENCE))
    q, k, v, hid = (to_dev_bf16(p[n]) for n in ("q_text", "k", "v", "hidden"))
    f.filter_layer(q, k, v, hid, to_dev(p["key_idx"]), to_dev(p["key_cnt"]), vis_cnt=to_dev(vis_cnt), want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    g, i = f.g.cpu().numpy(), f.i.cpu().numpy()
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    ho = bf16_bits(f.hidden_out)
    vs, N = w.vis_start, w.n_txt
    for b, m in enumerate(vis_cnt):
        lb = vs + int(m) + N
        G, I = oracle.score(p["q_text"][b:b + 1], p["k"][b:b + 1, :, :lb], vs, int(m), vs + int(m))
        assert_scores_close(g[b:b + 1, :m], G, "G")
        assert_scores_close(i[b:b + 1, :m], I, "I")
        # the selection is a function of its fp32 inputs: the oracle's rule on the GPU's own scores
        ref_idx, ref_cnt, _, _ = oracle.select(g[b:b + 1, :m].copy(), i[b:b + 1, :m].copy(), lb, p["key_idx"][b:b + 1],
                                               p["key_cnt"][b:b + 1], mode=oracle.MODE_THRESHOLD)
        n = int(ref_cnt[0])
        assert cnt[b] == n and 0 < n <= m
        assert np.array_equal(idx[b, :n], ref_idx[0, :n])
        rows = np.concatenate([np.arange(vs), vs + idx[b, :n], vs + m + np.arange(N)])
        assert np.array_equal(ho[b, :len(rows)], p["hidden"][b, rows])
    f.close()

"""GPU parity of the single-call filter (score, selection and gather in one launch where the
plan allows it) against the CPU oracle, and bit-equality with the three separate calls."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import build as md_build
from paper_2411_10803_b200 import synth

from parity_util import assert_kept_matches, bf16_bits, cfg, force, host_gather, to_dev, to_dev_bf16
from test_gpu_parity import key_args, run_chain_and_check, small

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    md_build.build()
    assert torch.cuda.is_available()


@pytest.fixture
def cluster(request, monkeypatch):
    force(monkeypatch, cluster=request.param)
    return request.param


def test_filter_tiny_reference_config_is_one_launch():
    run_chain_and_check(synth.WORKLOADS["c1_tiny"], path="filter", expect_launches=1)


def _skip_unless_fused(w):
    f = md.Filter(cfg(w))
    fused = f.score_variant == "fused_cluster_tcgen05"
    f.close()
    if not fused:
        pytest.skip("this shape does not fit the fused kernel at that cluster size")


@pytest.mark.parametrize("cluster", [0, 1, 2, 3, 5, 8, 11, 16], indirect=True)
def test_filter_small_ragged_batch(cluster):
    # 5 requests, ragged sizes, vision span not at 0, more kept rows than CTAs in the cluster
    w = small(batch=5, n_vis=333 if cluster != 1 else 270, n_txt=21, n_heads=3, hidden=384, key_cnt=9, budget=40,
              vis_start=2)
    _skip_unless_fused(w)
    run_chain_and_check(w, path="filter", expect_launches=1)


@pytest.mark.parametrize("cluster", [0, 4], indirect=True)
def test_filter_fewer_kept_rows_than_ctas(cluster):
    w = small(batch=3, n_vis=200, n_txt=9, key_cnt=1, budget=2)
    run_chain_and_check(w, path="filter", expect_launches=1)


def test_full_size_plans_are_single_launches():
    # (every request of these workloads is compared with the oracle, on this path too, by
    # test_full_config_every_request_matches_oracle)
    for name, launches in (("c2_llava7b_b16", 1), ("c2_llava7b_b64", 1), ("c3_next7b", 1), ("c5_13b_b64", 1),
                           ("c4_video", 1)):
        f = md.Filter(cfg(synth.WORKLOADS[name]))
        assert f.filter_launches == launches, name
        f.close()


def test_filter_falls_back_to_separate_launches_where_the_fused_geometry_does_not_fit():
    # 4000 vision tokens with 100 text rows exceed 16 CTAs x 160 keys: the call still does the whole step
    w = synth.WORKLOADS["c4_video"].with_(batch=1, n_vis=4000, n_txt=100, n_heads=2, hidden=256, budget=300)
    run_chain_and_check(w, path="filter", expect_launches=4)


def test_filter_video_runs_on_a_large_cluster_with_two_statistics_slots(monkeypatch):
    # (the planner prefers the two-pass kernel for this shape: force the fused one)
    force(monkeypatch, variant="fused")
    w = synth.WORKLOADS["c4_video"].with_(batch=2)
    run_chain_and_check(w, path="filter", expect_launches=1)


def test_filter_next7b_runs_on_a_cluster_of_more_than_eight(monkeypatch):
    # 2944 keys per request need more than 8 CTAs x 320 keys: non-portable cluster size, few statistics slots
    force(monkeypatch, variant="fused")
    w = synth.WORKLOADS["c3_next7b"].with_(batch=2)
    run_chain_and_check(w, path="filter", expect_launches=1)


def _run_both(w, monkeypatch, cfg_kw=None, drop=()):
    """The single call and the three calls on the same inputs -> two dicts of host arrays."""
    d = synth.make_batch(w)
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    out = []
    for staged in (False, True):
        force(monkeypatch, staged=staged)
        f = md.Filter(cfg(w, **(cfg_kw or {})))
        assert f.filter_launches == (3 if staged else 1)
        f.filter(q, k, None if "v" in drop else v, None if "hidden" in drop else hid, ki, kc, want_s=True)
        torch.cuda.synchronize()
        assert f.device_status() == (0, 0)
        out.append(dict(g=f.g.cpu().numpy(), i=f.i.cpu().numpy(), s=f.s.cpu().numpy(),
                        idx=f.kept_idx.cpu().numpy(), cnt=f.kept_cnt.cpu().numpy(), ho=bf16_bits(f.hidden_out),
                        ko=bf16_bits(f.k_out), vo=bf16_bits(f.v_out)))
        f.close()
    return d, out[0], out[1]


@pytest.mark.parametrize("mode_kw", [
    dict(),
    dict(mode=md.MUSTDROP_MODE_THRESHOLD),
    dict(criteria=md.MUSTDROP_CRIT_GLOBAL_ONLY),
    dict(criteria=md.MUSTDROP_CRIT_INDIVIDUAL_ONLY),
    dict(causal=0),
])
def test_filter_equals_the_three_calls_bit_for_bit(mode_kw, monkeypatch):
    w = small(batch=4, n_vis=777, n_txt=33, n_heads=5, hidden=640, key_cnt=11, budget=100)
    d, one, three = _run_both(w, monkeypatch, mode_kw)
    for name in ("g", "i", "s", "cnt"):
        assert np.array_equal(one[name], three[name]), name
    for b in range(w.batch):
        n = one["cnt"][b]
        assert np.array_equal(one["idx"][b, :n], three["idx"][b, :n])
        assert np.array_equal(one["ho"][b, :n], three["ho"][b, :n])
        assert np.array_equal(one["ko"][b, :, :n], three["ko"][b, :, :n])
        assert np.array_equal(one["vo"][b, :, :n], three["vo"][b, :, :n])
    if mode_kw.get("mode") == md.MUSTDROP_MODE_THRESHOLD:
        # the oracle's rule on the GPU's own scores: Eq. 9 and Eq. 10 as printed, key set kept
        ref_idx, ref_cnt, _, _ = oracle.select(one["g"], one["i"], w.seq_len, d["key_idx"], d["key_cnt"],
                                                mode=oracle.MODE_THRESHOLD)
        assert np.array_equal(ref_cnt, one["cnt"])
        for b in range(w.batch):
            assert np.array_equal(ref_idx[b, :ref_cnt[b]], one["idx"][b, :ref_cnt[b]])


@pytest.mark.parametrize("drop", [("v",), ("hidden",), ("v", "hidden")])
def test_filter_copies_only_the_tensors_it_is_given(drop, monkeypatch):
    w = small(batch=3, n_vis=300, n_txt=12, n_heads=4, hidden=512, key_cnt=5, budget=37)
    d, one, three = _run_both(w, monkeypatch, drop=drop)
    idx, cnt = one["idx"], one["cnt"]
    assert np.array_equal(idx, three["idx"]) and np.array_equal(cnt, three["cnt"])
    zh, zk, zv = np.zeros_like(one["ho"]), np.zeros_like(one["ko"]), np.zeros_like(one["vo"])
    eh, ek, ev = host_gather(idx, cnt, w.vis_start, d["hidden"], d["k"], d["v"], zh, zk, zv)
    assert np.array_equal(one["ko"], ek)
    # a tensor that was not given stays as allocated (zeros)
    assert np.array_equal(one["ho"], zh if "hidden" in drop else eh)
    assert np.array_equal(one["vo"], zv if "v" in drop else ev)


def test_filter_without_a_key_set_and_keep_all():
    w = small(batch=2, n_vis=130, n_txt=5, key_cnt=0, budget=130)
    run_chain_and_check(w, path="filter", expect_launches=1)


def test_filter_is_deterministic_and_repeatable_on_one_stream():
    w = synth.WORKLOADS["c2_llava7b_b16"].with_(batch=6)
    d = synth.make_batch(w)
    f = md.Filter(cfg(w))
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    f.filter(q, k, v, hid, ki, kc)
    first = (f.g.clone(), f.i.clone(), f.kept_idx.clone(), f.hidden_out.clone(), f.k_out.clone(), f.v_out.clone())
    for _ in range(5):   # back to back: each launch overlaps the tail of the one before
        f.filter(q, k, v, hid, ki, kc)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    now = (f.g, f.i, f.kept_idx, f.hidden_out, f.k_out, f.v_out)
    for a, b in zip(first, now):
        assert torch.equal(a, b)
    f.close()


# ---- more than 64 text rows scored by two launches over the same keys ---------------------------

@pytest.mark.parametrize("n_txt,causal", [(65, 1), (96, 1), (128, 1), (100, 0)])
def test_row_split_score_and_filter_match_oracle(n_txt, causal, monkeypatch):
    force(monkeypatch, variant="row_split")
    w = small(batch=3, n_vis=500, n_txt=n_txt, n_heads=3, hidden=384, key_cnt=7, budget=60, vis_start=1)
    d = synth.make_batch(w)
    f = md.Filter(cfg(w, causal=causal))
    assert "two launches" in f.description and f.filter_launches == 2
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    # the score call alone (two launches, the second combining), then the whole step
    f.score(q, k)
    torch.cuda.synchronize()
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start, causal=bool(causal))
    from parity_util import assert_scores_close
    assert_scores_close(f.g.cpu().numpy(), G, "G")
    assert_scores_close(f.i.cpu().numpy(), I, "I")
    f.g.zero_(); f.i.zero_()
    f.filter(q, k, v, hid, ki, kc, want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    assert_scores_close(f.g.cpu().numpy(), G, "G")
    assert_scores_close(f.i.cpu().numpy(), I, "I")
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, w.seq_len, d["key_idx"], d["key_cnt"], budget=w.budget)
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, d["key_idx"], d["key_cnt"])
    zh, zk, zv = (np.zeros_like(bf16_bits(t)) for t in (f.hidden_out, f.k_out, f.v_out))
    eh, ek, ev = host_gather(idx, cnt, w.vis_start, d["hidden"], d["k"], d["v"], zh, zk, zv)
    assert np.array_equal(bf16_bits(f.hidden_out), eh) and np.array_equal(bf16_bits(f.k_out), ek)
    assert np.array_equal(bf16_bits(f.v_out), ev)
    f.close()


# ---- bounded waits: a wait that runs out is reported, not a hang ---------------------------------

@pytest.mark.parametrize("grid_ctas", [2, 4, 6])
def test_filter_on_a_grid_plan(grid_ctas, monkeypatch):
    """The request's CTAs as ordinary CTAs of the grid: statistics and the barrier before the
    selection go through counters in global memory, which every call leaves at zero - so the
    same plan and workspace are used three times in a row."""
    force(monkeypatch, variant="grid", cluster=grid_ctas)
    w = small(batch=5, n_vis=333, n_txt=21, n_heads=3, hidden=384, key_cnt=9, budget=40, vis_start=2)
    f = md.Filter(cfg(w))
    assert "grid plan" in f.description and f.filter_launches == 1
    f.close()
    run_chain_and_check(w, path="filter", expect_launches=1)
    run_chain_and_check(w, path="staged")
    d = synth.make_batch(w)
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    f = md.Filter(cfg(w))
    f.filter(q, k, v, hid, ki, kc)
    first = (f.g.clone(), f.i.clone(), f.kept_idx.clone(), f.hidden_out.clone(), f.k_out.clone())
    for _ in range(3):
        f.filter(q, k, v, hid, ki, kc)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    for a, b in zip(first, (f.g, f.i, f.kept_idx, f.hidden_out, f.k_out)):
        assert torch.equal(a, b)
    f.close()


@pytest.mark.parametrize("cluster", [0, 3], indirect=True)
def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_unaffected(cluster):
    """The configuration's debug_wait_cycles shortens the waits between the kernel's warp roles to
    a few cycles, so the first wait for a copy from global memory runs out: the kernel must come
    back by itself, report MUSTDROP_ERR_TIMEOUT, mark every request invalid (kept_cnt = -1) and
    leave the device usable - the same step with normal waits, run right behind it on the same
    stream, gives the oracle's result."""
    w = small(batch=3, n_vis=333, n_txt=21, n_heads=3, hidden=384, key_cnt=9, budget=40, vis_start=2)
    d = synth.make_batch(w)
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    bad = md.Filter(cfg(w, debug_wait_cycles=64))
    assert bad.filter_launches == 1
    bad.kept_cnt.fill_(7)
    bad.filter(q, k, v, hid, ki, kc)
    good = md.Filter(cfg(w))
    good.filter(q, k, v, hid, ki, kc, want_s=True)
    torch.cuda.synchronize()
    code, _ = bad.device_status()
    assert code == md.MUSTDROP_ERR_TIMEOUT
    assert (bad.kept_cnt.cpu().numpy() == -1).all()
    assert good.device_status() == (0, 0)
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, w.seq_len, d["key_idx"], d["key_cnt"], budget=w.budget)
    idx, cnt = good.kept_idx.cpu().numpy(), good.kept_cnt.cpu().numpy()
    assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, d["key_idx"], d["key_cnt"])
    rh, rk, rv = oracle.compact(idx, cnt, w.vis_start, d["hidden"], d["k"], d["v"])
    assert np.array_equal(bf16_bits(good.hidden_out), rh) and np.array_equal(bf16_bits(good.k_out), rk)
    assert np.array_equal(bf16_bits(good.v_out), rv)
    # the score-only call gives up the same way (status word only: it has no kept_cnt)
    bad.workspace.zero_()
    bad.score(q, k)
    torch.cuda.synchronize()
    assert bad.device_status()[0] == md.MUSTDROP_ERR_TIMEOUT
    bad.close()
    good.close()


def test_compact_skips_a_request_marked_invalid():
    """kept_cnt = -1 (a request whose selection failed) and a count beyond the capacity: nothing is
    written for the first, the second is clamped; both are recorded; nothing lands outside the outputs."""
    w = small(batch=3, n_vis=50, n_txt=6, n_heads=2, hidden=256, key_cnt=0, budget=8, vis_start=1)
    d = synth.make_batch(w)
    f = md.Filter(cfg(w, flags=md.MUSTDROP_FLAG_REBUILD_SEQUENCE))
    kept = np.tile(np.arange(8, dtype=np.int32), (3, 1))
    cnt = np.array([-1, 8, 99], np.int32)
    for t in (f.hidden_out, f.k_out, f.v_out):
        t.fill_(-3.0)                                            # canary value in every output row
    f.compact(to_dev_bf16(d["hidden"]), to_dev_bf16(d["k"]), to_dev_bf16(d["v"]), to_dev(kept), to_dev(cnt))
    torch.cuda.synchronize()
    canary = bf16_bits(torch.full((1,), -3.0, dtype=torch.bfloat16, device="cuda"))[0]
    ho, ko = bf16_bits(f.hidden_out), bf16_bits(f.k_out)
    assert (ho[0] == canary).all() and (ko[0] == canary).all()   # the invalid request: untouched
    rows = np.concatenate([np.arange(1), 1 + kept[1], 1 + 50 + np.arange(6)])
    for b in (1, 2):                                             # 99 is clamped to the capacity of 8
        assert np.array_equal(ho[b, :len(rows)], d["hidden"][b, rows])
        assert np.array_equal(ko[b][:, :len(rows)], d["k"][b][:, rows])
    assert f.device_status()[0] == md.MUSTDROP_ERR_BAD_KEY_INDEX
    f.close()

"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Stage-isolated first (each kernel fed the oracle's inputs), then the chain."""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import build as md_build
from paper_2411_10803_b200 import synth

from parity_util import (assert_kept_matches, assert_scores_close, bf16_bits, cfg, force, full_config_reference,
                         host_gather, oracle_scores_all_requests, to_dev, to_dev_bf16)

pytestmark = pytest.mark.gpu

TINY = synth.WORKLOADS["c1_tiny"]


@pytest.fixture(scope="module", autouse=True)
def _built():
    md_build.build()
    assert torch.cuda.is_available()


def small(**kw):
    base = dict(batch=2, n_vis=100, n_txt=7, n_heads=3, hidden=384, n_salient=3, key_cnt=4, budget=16)
    base.update(kw)
    return TINY.with_(**base)


VARIANTS = ["auto", "two_pass", "fused:1", "fused:2", "fused:3", "fused:5", "fused:8", "fused:12", "fused:16",
            "grid:2", "grid:3", "grid:7", "grid:24"]      # grid: CTAs per request of a plan without clusters


@pytest.fixture
def variant(request, monkeypatch):
    """Force a score kernel variant / cluster size through the configuration's debugging overrides."""
    v = request.param
    if v == "two_pass":
        force(monkeypatch, variant="two_pass")
    elif v.startswith("fused:"):
        force(monkeypatch, variant="fused", cluster=v.split(":")[1])
    elif v.startswith("grid:"):
        force(monkeypatch, variant="grid", cluster=v.split(":")[1])
    return v


def check_variant(f, v):
    if v == "two_pass":
        assert f.score_variant == "two_pass_mma"
    elif v.startswith("fused:") and f.score_variant != "fused_cluster_tcgen05":
        f.close()
        pytest.skip("this shape does not fit the fused kernel at that cluster size")
    elif v.startswith("grid:") and "grid plan" not in f.description:
        f.close()
        pytest.skip("this shape has no plan with that many CTAs per request")


def key_args(w, d):
    if w.key_cnt == 0:
        return None, None
    return to_dev(d["key_idx"]), to_dev(d["key_cnt"])


# ---- score -----------------------------------------------------------------------------------

SCORE_CASES = [
    dict(),                                                      # ragged everything
    dict(n_vis=1, n_txt=1, n_heads=1, hidden=128, n_salient=0, key_cnt=0, budget=1),
    dict(n_vis=17, n_txt=16, n_salient=2),
    dict(n_vis=64, n_txt=32, n_heads=2, hidden=256),
    dict(n_vis=129, n_txt=33, vis_start=5),
    dict(n_vis=200, n_txt=64, n_heads=5, hidden=640),
    dict(n_vis=300, n_txt=100, n_heads=2, hidden=256, vis_start=3),
    dict(n_vis=576, n_txt=128, n_heads=2, hidden=256, batch=1),
    dict(n_vis=700, n_txt=96, n_heads=1, hidden=128, batch=3),
]


@pytest.mark.parametrize("variant", VARIANTS, indirect=True)
@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("case", range(len(SCORE_CASES)))
def test_score_matches_oracle(case, causal, variant):
    w = small(**SCORE_CASES[case])
    d = synth.make_batch(w, with_values=False)
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start, bool(causal))
    f = md.Filter(cfg(w, causal=causal))
    check_variant(f, variant)
    g, i = f.score(to_dev_bf16(d["q_text"]), to_dev_bf16(d["k"]))
    torch.cuda.synchronize()
    assert_scores_close(g.cpu().numpy(), G, "G case %d" % case)
    assert_scores_close(i.cpu().numpy(), I, "I case %d" % case)
    assert f.device_status() == (0, 0)
    f.close()


@pytest.mark.parametrize("variant", ["auto", "two_pass", "fused:2"], indirect=True)
def test_score_with_text_after_the_span_and_explicit_scale(variant):
    """Keys beyond the text span (a later turn) are visible only when the mask is off."""
    w = small(n_vis=90, n_txt=9)
    d = synth.make_batch(w, with_values=False)
    extra = 11
    rng = np.random.default_rng(3)
    tail = synth.f32_to_bf16_bits(rng.standard_normal((w.batch, w.n_heads, extra, 128), dtype=np.float32))
    k = np.concatenate([d["k"], tail], axis=2)
    for causal in (1, 0):
        G, I = oracle.score(d["q_text"], k, w.vis_start, w.n_vis, w.txt_start, bool(causal), scale=0.05)
        f = md.Filter(cfg(w, causal=causal, seq_len=w.seq_len + extra, scale=0.05))
        g, i = f.score(to_dev_bf16(d["q_text"]), to_dev_bf16(k))
        assert_scores_close(g.cpu().numpy(), G)
        assert_scores_close(i.cpu().numpy(), I)
        f.close()


@pytest.mark.parametrize("variant", ["auto", "two_pass", "fused:2"], indirect=True)
def test_score_with_strided_keys(variant):
    """K stored as [B, L, H, D] (token-major) and addressed through the plan's strides."""
    w = small(n_vis=70, n_txt=12, n_heads=4, hidden=512)
    d = synth.make_batch(w, with_values=False)
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    k_tok_major = np.ascontiguousarray(d["k"].transpose(0, 2, 1, 3))           # [B,L,H,D]
    H, L, D = w.n_heads, w.seq_len, 128
    f = md.Filter(cfg(w, k_stride_b=L * H * D, k_stride_h=D, k_stride_l=H * D))
    g, i = f.score(to_dev_bf16(d["q_text"]), to_dev_bf16(k_tok_major))
    assert_scores_close(g.cpu().numpy(), G)
    assert_scores_close(i.cpu().numpy(), I)
    f.close()


@pytest.mark.parametrize("variant", ["auto", "two_pass", "fused:2"], indirect=True)
def test_score_extreme_logits_do_not_overflow(variant):
    w = small(n_vis=40, n_txt=6, n_heads=2, hidden=256, n_salient=0)
    d = synth.make_batch(w, with_values=False)
    q = synth.bf16_bits_to_f32(d["q_text"]) * 6.0
    k = synth.bf16_bits_to_f32(d["k"]) * 6.0            # logits of a few hundred
    qb, kb = synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k)
    G, I = oracle.score(qb, kb, w.vis_start, w.n_vis, w.txt_start)
    f = md.Filter(cfg(w))
    g, i = f.score(to_dev_bf16(qb), to_dev_bf16(kb))
    g, i = g.cpu().numpy(), i.cpu().numpy()
    assert np.isfinite(g).all() and np.isfinite(i).all()
    big = G > 1e-6                                       # compare where the mass is; the rest underflows alike
    assert_scores_close(g[big], G[big])
    assert_scores_close(i[big], I[big])
    f.close()


@pytest.mark.parametrize("variant", ["auto", "fused:1", "fused:2", "fused:5", "fused:12"], indirect=True)
@pytest.mark.parametrize("n_txt", [20, 100])
def test_score_with_logits_that_grow_along_the_keys(n_txt, variant):
    """Later keys carry ever larger logits, so the stabiliser an exp warp takes from the first
    columns it sees falls short by far more than 2^32 and the already stored exponentials have to
    be rescaled (several times per row)."""
    w = small(batch=2, n_vis=700, n_txt=n_txt, n_heads=2, hidden=256, n_salient=0)
    d = synth.make_batch(w, with_values=False)
    q = synth.bf16_bits_to_f32(d["q_text"])
    k = synth.bf16_bits_to_f32(d["k"])
    u = q.mean(axis=2, keepdims=True)                                    # [B,H,1,D] mean text query
    u /= np.linalg.norm(u, axis=-1, keepdims=True)
    ramp = np.linspace(0.0, 180.0, w.seq_len, dtype=np.float32)[None, None, :, None]
    k = k + ramp * u * np.sqrt(128.0) / np.maximum(np.linalg.norm(q, axis=-1).mean(), 1e-6) * 3.0
    qb, kb = synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k.astype(np.float32))
    G, I = oracle.score(qb, kb, w.vis_start, w.n_vis, w.txt_start)
    f = md.Filter(cfg(w))
    check_variant(f, variant)
    g, i = f.score(to_dev_bf16(qb), to_dev_bf16(kb))
    torch.cuda.synchronize()
    g, i = g.cpu().numpy(), i.cpu().numpy()
    assert f.device_status() == (0, 0)
    assert np.isfinite(g).all() and np.isfinite(i).all()
    big = G > 1e-12
    assert big.sum() > 10
    assert_scores_close(g[big], G[big], "G")
    assert_scores_close(i[big], I[big], "I")
    assert (g[~big] <= 1e-9).all()
    f.close()


# ---- select ----------------------------------------------------------------------------------

def _random_scores(seed, B, M, N=9):
    rng = np.random.default_rng(seed)
    a = rng.random((B, N, M)) ** 4 / M
    return a.sum(1).astype(np.float32), a.max(1).astype(np.float32)


@pytest.mark.parametrize("M,key_max,budgets", [
    (1, 0, [1]), (17, 3, [3, 4, 16, 17]), (576, 32, [32, 64, 128, 192, 575, 576]),
    (2880, 64, [64, 320, 2879]), (4096, 0, [1, 2048, 4096]), (1000, 1000, [1000]),
])
@pytest.mark.parametrize("criteria", [md.MUSTDROP_CRIT_DUAL, md.MUSTDROP_CRIT_GLOBAL_ONLY,
                                      md.MUSTDROP_CRIT_INDIVIDUAL_ONLY])
def test_select_budget_is_bit_exact_given_oracle_scores(M, key_max, budgets, criteria):
    B = 3
    G, I = _random_scores(M + key_max, B, M)
    rng = np.random.default_rng(M)
    if key_max:
        key_idx = np.stack([rng.choice(M, key_max, replace=False) for _ in range(B)]).astype(np.int32)
        key_cnt = np.array([key_max, key_max // 2, 0], np.int32)
    else:
        key_idx = key_cnt = None
    for budget in budgets:
        ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, M + 9, key_idx, key_cnt, criteria=criteria, budget=budget)
        w = small(batch=B, n_vis=M, n_txt=9, key_cnt=key_max, budget=budget)
        f = md.Filter(cfg(w, criteria=criteria))
        f.select(None if key_idx is None else to_dev(key_idx), None if key_cnt is None else to_dev(key_cnt),
                 g=to_dev(G), i=to_dev(I))
        idx, cnt, s = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy(), f.s.cpu().numpy()
        assert np.array_equal(s, ref_s)
        assert np.array_equal(cnt, ref_cnt)
        assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, key_idx, key_cnt, exact=True)
        f.close()


def test_select_ties_take_the_lower_index():
    B, M = 2, 300
    G, I = _random_scores(5, B, M)
    G[:, 50:250] = G[:, 50:51]              # two hundred equal scores straddling every cut
    I[:, 50:250] = I[:, 50:51]
    for budget in (10, 60, 150, 260):
        ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, M + 9, budget=budget)
        w = small(batch=B, n_vis=M, n_txt=9, key_cnt=0, budget=budget)
        f = md.Filter(cfg(w))
        f.select(g=to_dev(G), i=to_dev(I))
        assert_kept_matches(f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy(), ref_idx, ref_cnt, ref_s, exact=True)
        f.close()


@pytest.mark.parametrize("criteria", [md.MUSTDROP_CRIT_DUAL, md.MUSTDROP_CRIT_GLOBAL_ONLY,
                                      md.MUSTDROP_CRIT_INDIVIDUAL_ONLY])
def test_select_threshold_mode_is_bit_exact(criteria):
    B, M = 4, 777
    G, I = _random_scores(11, B, M)
    rng = np.random.default_rng(2)
    key_idx = np.stack([rng.choice(M, 20, replace=False) for _ in range(B)]).astype(np.int32)
    key_cnt = np.array([20, 0, 7, 20], np.int32)
    gamma, alpha = 1.1 / M, float(np.median(I))
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, M + 9, key_idx, key_cnt, mode=oracle.MODE_THRESHOLD,
                                               criteria=criteria, gamma=gamma, alpha=alpha)
    assert len(set(ref_cnt.tolist())) > 1                  # the kept count differs per request
    w = small(batch=B, n_vis=M, n_txt=9, key_cnt=20, budget=0)
    f = md.Filter(cfg(w, mode=md.MUSTDROP_MODE_THRESHOLD, criteria=criteria, gamma=gamma, alpha=alpha))
    f.select(to_dev(key_idx), to_dev(key_cnt), g=to_dev(G), i=to_dev(I))
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, key_idx, key_cnt, exact=True)
    for b in range(B):                                       # slots past the count stay untouched
        assert (idx[b, cnt[b]:] == -1).all()
    f.close()


def test_select_ignores_bad_and_repeated_key_indices_and_reports_them():
    B, M = 2, 64
    G, I = _random_scores(7, B, M)
    key_idx = np.array([[3, 3, -1, 99, 7, 7, 0, 0], [5, 6, 7, 8, 9, 10, 11, 12]], np.int32)
    key_cnt = np.array([8, 8], np.int32)
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, M + 9, key_idx, key_cnt, budget=10)
    w = small(batch=B, n_vis=M, n_txt=9, key_cnt=8, budget=10)
    f = md.Filter(cfg(w))
    assert f.device_status() == (0, 0)
    f.select(to_dev(key_idx), to_dev(key_cnt), g=to_dev(G), i=to_dev(I))
    assert_kept_matches(f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy(), ref_idx, ref_cnt, ref_s, exact=True)
    code, detail = f.device_status()
    assert code == md.MUSTDROP_ERR_BAD_KEY_INDEX and detail in (2, 3)    # request 0, slot 2 or 3
    f.close()


# ---- compact ---------------------------------------------------------------------------------

@pytest.mark.parametrize("kw", [dict(), dict(vis_start=6), dict(n_heads=1, hidden=128),
                                dict(n_heads=5, hidden=1000, n_vis=33, budget=33)])
def test_compact_is_byte_exact_given_oracle_indices(kw):
    w = small(**kw)
    d = synth.make_batch(w)
    rng = np.random.default_rng(1)
    cap = w.budget
    kept = np.stack([np.sort(rng.choice(w.n_vis, cap, replace=False)) for _ in range(w.batch)]).astype(np.int32)
    cnt = np.array([cap, max(cap - 5, 0)][: w.batch], np.int32)
    ho, ko, vo = oracle.compact(kept, cnt, w.vis_start, d["hidden"], d["k"], d["v"], fill=0)
    f = md.Filter(cfg(w))
    f.compact(to_dev_bf16(d["hidden"]), to_dev_bf16(d["k"]), to_dev_bf16(d["v"]), to_dev(kept), to_dev(cnt))
    assert np.array_equal(bf16_bits(f.hidden_out), ho)
    assert np.array_equal(bf16_bits(f.k_out), ko)
    assert np.array_equal(bf16_bits(f.v_out), vo)
    f.close()


def test_compact_keep_all_is_the_identity_and_strides_work():
    w = small(n_vis=40, n_txt=5, budget=40, key_cnt=0, n_heads=4, hidden=512)
    d = synth.make_batch(w)
    M, H, L, D = w.n_vis, w.n_heads, w.seq_len, 128
    kept = np.tile(np.arange(M, dtype=np.int32), (w.batch, 1))
    cnt = np.full((w.batch,), M, np.int32)
    # K and V stored token-major [B,L,H,D]
    f = md.Filter(cfg(w, k_stride_b=L * H * D, k_stride_h=D, k_stride_l=H * D,
                                v_stride_b=L * H * D, v_stride_h=D, v_stride_l=H * D))
    kt = np.ascontiguousarray(d["k"].transpose(0, 2, 1, 3))
    vt = np.ascontiguousarray(d["v"].transpose(0, 2, 1, 3))
    f.compact(to_dev_bf16(d["hidden"]), to_dev_bf16(kt), to_dev_bf16(vt), to_dev(kept), to_dev(cnt))
    assert np.array_equal(bf16_bits(f.hidden_out), d["hidden"][:, :M])
    assert np.array_equal(bf16_bits(f.k_out), d["k"][:, :, :M])
    assert np.array_equal(bf16_bits(f.v_out), d["v"][:, :, :M])
    f.close()


def test_compact_skips_an_out_of_range_index_and_reports_it():
    w = small(n_vis=20, n_txt=4, budget=4, key_cnt=0)
    d = synth.make_batch(w)
    kept = np.array([[1, 2, 77, 5], [0, 1, 2, 3]], np.int32)
    cnt = np.array([4, 4], np.int32)
    f = md.Filter(cfg(w))
    f.compact(to_dev_bf16(d["hidden"]), None, None, to_dev(kept), to_dev(cnt))
    out = bf16_bits(f.hidden_out)
    assert np.array_equal(out[0, 1], d["hidden"][0, 2]) and (out[0, 2] == 0).all()
    code, _ = f.device_status()
    assert code == md.MUSTDROP_ERR_BAD_KEY_INDEX
    f.close()


# ---- the chain -------------------------------------------------------------------------------

def run_chain_and_check(w, check_scores=True, path="staged", expect_launches=None, ref=None):
    """score -> select -> compact on the GPU for the whole batch (three calls, or the single
    mustdrop_filter call with path="filter"), compared with the oracle on EVERY request.
    ref = (inputs, G, I) when the oracle's scores of the batch are already at hand."""
    if ref is None:
        d = synth.make_batch(w)
        G, I = oracle_scores_all_requests(d, w)
    else:
        d, G, I = ref
    f = md.Filter(cfg(w))
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    if path == "filter":
        if expect_launches is not None:
            assert f.filter_launches == expect_launches
        f.filter(q, k, v, hid, ki, kc, want_s=True)
    else:
        f.run(q, k, v, hid, ki, kc, want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    g, i = f.g.cpu().numpy(), f.i.cpu().numpy()
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    ho, ko, vo = bf16_bits(f.hidden_out), bf16_bits(f.k_out), bf16_bits(f.v_out)
    del q, k, v, hid
    assert (cnt == w.budget).all()
    if check_scores:
        assert_scores_close(g, G, "G")
        assert_scores_close(i, I, "I")
    kidx = d["key_idx"] if w.key_cnt else None
    kcnt = d["key_cnt"] if w.key_cnt else None
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, w.seq_len, kidx, kcnt, budget=w.budget)
    swapped = assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, kidx, kcnt)
    # the compacted tensors against the oracle's, byte for byte, request by request; a request
    # whose kept set differs inside the near-tie window is compared with the oracle's gather of
    # the GPU's own (valid) indices instead
    n_exact = 0
    for b in range(w.batch):
        same = np.array_equal(idx[b, :cnt[b]], ref_idx[b, :ref_cnt[b]])
        n_exact += int(same)
        use_idx = ref_idx[b:b + 1] if same else idx[b:b + 1]
        rh, rk, rv = oracle.compact(use_idx, cnt[b:b + 1], w.vis_start, d["hidden"][b:b + 1], d["k"][b:b + 1],
                                    d["v"][b:b + 1])
        assert np.array_equal(ho[b], rh[0]) and np.array_equal(ko[b], rk[0]) and np.array_equal(vo[b], rv[0]), b
    print("%s / %s: %d of %d requests bit-exact, %d near-tie swaps" % (w.name, path, n_exact, w.batch, swapped))
    # planted salient keys are retained (they dominate both criteria)
    if w.n_salient:
        for b in range(w.batch):
            kept = set(idx[b, :cnt[b]].tolist())
            hit = len(kept & set(d["salient_idx"][b].tolist()))
            assert hit >= min(w.n_salient, w.budget - w.key_cnt) * 0.9
    f.close()
    return swapped


def test_chain_tiny_reference_config():
    run_chain_and_check(synth.WORKLOADS["c1_tiny"])


def test_chain_small_ragged_batch():
    run_chain_and_check(small(batch=5, n_vis=333, n_txt=21, n_heads=3, hidden=384, key_cnt=9, budget=40, vis_start=2))


# ---- the five listed configurations at full size: every request against the oracle, both paths ----

FULL_CONFIGS = [("c1_tiny", None), ("c2_llava7b_b16", 192), ("c2_llava7b_b16", 128), ("c2_llava7b_b16", 64),
                ("c2_llava7b_b64", None), ("c3_next7b", None), ("c4_video", None), ("c5_13b_b64", None)]


@pytest.mark.parametrize("path", ["staged", "filter"])
@pytest.mark.parametrize("name,budget", FULL_CONFIGS)
def test_full_config_every_request_matches_oracle(name, budget, path):
    w, d, G, I = full_config_reference(name)     # the oracle's scores: once per workload, shared by the paths
    if budget is not None:
        w = w.with_(budget=budget)
    run_chain_and_check(w, path=path, ref=(d, G, I))


def test_chain_is_deterministic():
    w = synth.WORKLOADS["c2_llava7b_b16"].with_(batch=4)
    d = synth.make_batch(w)
    f = md.Filter(cfg(w))
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    f.run(q, k, v, hid, ki, kc)
    a = (f.g.clone(), f.i.clone(), f.kept_idx.clone(), f.hidden_out.clone())
    f.run(q, k, v, hid, ki, kc)
    torch.cuda.synchronize()
    assert torch.equal(a[0], f.g) and torch.equal(a[1], f.i) and torch.equal(a[2], f.kept_idx)
    assert torch.equal(a[3], f.hidden_out)
    f.close()


# ---- the per-head reading of Eq. 10 (MUSTDROP_FLAG_PER_HEAD_MAX) ------------------------------------

@pytest.mark.parametrize("variant", VARIANTS, indirect=True)
@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("kw", [dict(), dict(batch=3, n_vis=333, n_txt=21, n_heads=5, hidden=640, vis_start=2),
                                dict(batch=2, n_vis=130, n_txt=100, n_heads=2, hidden=256),
                                dict(batch=2, n_vis=700, n_txt=64, n_heads=4, hidden=512)])
def test_score_per_head_max_matches_oracle(kw, causal, variant):
    w = small(**kw)
    d = synth.make_batch(w, with_values=False)
    f = md.Filter(cfg(w, causal=causal, flags=md.MUSTDROP_FLAG_PER_HEAD_MAX))
    check_variant(f, variant)
    if variant == "auto":
        assert f.score_variant == "fused_cluster_tcgen05"      # the flag runs on the one-pass kernel
    f.score(to_dev_bf16(d["q_text"]), to_dev_bf16(d["k"]))
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    G, I = oracle.score_per_head(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start, causal=bool(causal))
    assert_scores_close(f.g.cpu().numpy(), G, "G")
    assert_scores_close(f.i.cpu().numpy(), I, "I (per head)")
    # and it is not the other reading
    _, I_mean_first = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start, causal=bool(causal))
    if w.n_heads > 1:
        assert np.any(np.abs(f.i.cpu().numpy() - I_mean_first) > 1e-2 * I_mean_first)
    f.close()


def test_per_head_max_at_the_batch64_shape_runs_the_one_launch_filter():
    w = synth.WORKLOADS["c2_llava7b_b64"].with_(batch=8)
    d = synth.make_batch(w)
    f = md.Filter(cfg(w, flags=md.MUSTDROP_FLAG_PER_HEAD_MAX))
    assert f.score_variant == "fused_cluster_tcgen05" and f.filter_launches == 1
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    f.filter(q, k, v, hid, ki, kc, want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    G, I = oracle_scores_all_requests(d, w, per_head=True)
    assert_scores_close(f.g.cpu().numpy(), G, "G")
    assert_scores_close(f.i.cpu().numpy(), I, "I (per head)")
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, w.seq_len, d["key_idx"], d["key_cnt"], budget=w.budget)
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, d["key_idx"], d["key_cnt"])
    rh, rk, rv = oracle.compact(idx, cnt, w.vis_start, d["hidden"], d["k"], d["v"])
    assert np.array_equal(bf16_bits(f.hidden_out), rh) and np.array_equal(bf16_bits(f.k_out), rk)
    assert np.array_equal(bf16_bits(f.v_out), rv)
    f.close()


def test_filter_call_with_per_head_max_selects_by_the_per_head_scores():
    w = synth.WORKLOADS["c2_llava7b_b16"].with_(batch=3)
    d = synth.make_batch(w)
    f = md.Filter(cfg(w, flags=md.MUSTDROP_FLAG_PER_HEAD_MAX))
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    ki, kc = key_args(w, d)
    f.filter(q, k, v, hid, ki, kc, want_s=True)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    G, I = oracle.score_per_head(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    ref_idx, ref_cnt, ref_s, _ = oracle.select(G, I, w.seq_len, d["key_idx"], d["key_cnt"], budget=w.budget)
    idx, cnt = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    assert_kept_matches(idx, cnt, ref_idx, ref_cnt, ref_s, d["key_idx"], d["key_cnt"])
    zh, zk, zv = (np.zeros_like(bf16_bits(t)) for t in (f.hidden_out, f.k_out, f.v_out))
    eh, ek, ev = host_gather(idx, cnt, w.vis_start, d["hidden"], d["k"], d["v"], zh, zk, zv)
    assert np.array_equal(bf16_bits(f.hidden_out), eh) and np.array_equal(bf16_bits(f.k_out), ek)
    assert np.array_equal(bf16_bits(f.v_out), ev)
    f.close()

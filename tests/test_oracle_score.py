"""Pins for the oracle's attention / importance-score functions (Eq. 1, Eq. 8, Eq. 10).

Each test fixes the oracle to something other than itself: a library softmax in float64,
closed forms, hand-computed rank-one logits, inequalities and equivariances.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2411_10803_b200 import synth


def _rand_case(seed, H=3, N=5, M=11, vis_start=2, D=16, extra_txt=0):
    rng = np.random.default_rng(seed)
    L = vis_start + M + N + extra_txt
    q = synth.f32_to_bf16_bits(rng.standard_normal((1, H, N, D), dtype=np.float32))
    k = synth.f32_to_bf16_bits(rng.standard_normal((1, H, L, D), dtype=np.float32))
    return q, k, vis_start, M, vis_start + M, L


def _torch_reference(q, k, vis_start, M, txt_start, causal, scale=None):
    """Independent float64 restatement with library routines (matmul + softmax)."""
    qd = torch.from_numpy(synth.bf16_bits_to_f64(q))
    kd = torch.from_numpy(synth.bf16_bits_to_f64(k))
    B, H, N, D = qd.shape
    L = kd.shape[2]
    scale = 1.0 / math.sqrt(D) if scale is None else scale
    z = torch.matmul(qd, kd.transpose(-1, -2)) * scale                      # [B,H,N,L]
    if causal:
        pos = txt_start + torch.arange(N).view(N, 1)
        mask = torch.arange(L).view(1, L) > pos
        z = z.masked_fill(mask, float("-inf"))
    p = torch.softmax(z, dim=-1)
    a = p.mean(dim=1)[:, :, vis_start:vis_start + M]                        # [B,N,M]
    return p.numpy(), a.sum(dim=1).numpy(), a.max(dim=1).values.numpy(), a.numpy()


@pytest.mark.parametrize("causal", [True, False])
def test_rows_sum_to_one_and_mask(causal):
    q, k, vs, M, ts, L = _rand_case(1)
    p = oracle.attention(q[0], k[0], ts, causal)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-12)
    assert (p >= 0).all()
    if causal:
        for i in range(q.shape[2]):
            assert (p[:, i, ts + i + 1:] == 0).all()
            assert (p[:, i, :ts + i + 1] > 0).all()
    else:
        assert (p > 0).all()


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("seed,vis_start,extra", [(2, 0, 0), (3, 4, 0), (4, 1, 3)])
def test_matches_library_softmax_float64(causal, seed, vis_start, extra):
    q, k, vs, M, ts, L = _rand_case(seed, vis_start=vis_start, extra_txt=extra)
    G, I, a = oracle.score(q, k, vs, M, ts, causal, return_a=True)
    p_ref, g_ref, i_ref, a_ref = _torch_reference(q, k, vs, M, ts, causal)
    p = oracle.attention(q[0], k[0], ts, causal)
    assert np.allclose(p, p_ref[0], rtol=1e-12, atol=1e-15)
    assert np.allclose(a, a_ref, rtol=1e-12, atol=1e-15)
    assert np.array_equal(G, g_ref.astype(np.float32))
    assert np.array_equal(I, i_ref.astype(np.float32))


def test_explicit_scale_is_used():
    q, k, vs, M, ts, L = _rand_case(5)
    G, I = oracle.score(q, k, vs, M, ts, True, scale=0.37)
    _, g_ref, i_ref, _ = _torch_reference(q, k, vs, M, ts, True, scale=0.37)
    assert np.allclose(G, g_ref, rtol=1e-6) and np.allclose(I, i_ref, rtol=1e-6)
    G0, _ = oracle.score(q, k, vs, M, ts, True)
    assert not np.allclose(G, G0, rtol=1e-3)


@pytest.mark.parametrize("causal", [True, False])
def test_identical_keys_closed_form(causal):
    """All keys equal => uniform attention over the visible keys."""
    H, N, M, D, vs = 2, 6, 9, 8, 3
    L = vs + M + N
    ts = vs + M
    rng = np.random.default_rng(7)
    q = synth.f32_to_bf16_bits(rng.standard_normal((1, H, N, D), dtype=np.float32))
    krow = synth.f32_to_bf16_bits(rng.standard_normal((D,), dtype=np.float32))
    k = np.broadcast_to(krow, (1, H, L, D)).copy()
    G, I = oracle.score(q, k, vs, M, ts, causal)
    if causal:
        g = sum(1.0 / (ts + i + 1) for i in range(N))      # a harmonic-number difference
        mx = 1.0 / (ts + 1)
    else:
        g, mx = N / L, 1.0 / L
    assert np.allclose(G, g, rtol=1e-6) and np.allclose(I, mx, rtol=1e-6)


def test_one_dominant_key():
    """A key whose logit exceeds all others by ~40 takes all the attention."""
    H, N, M, D = 2, 4, 7, 16
    ts, L = M, M + N
    q = np.zeros((1, H, N, D), np.float32)
    q[..., 0] = 8.0
    k = np.zeros((1, H, L, D), np.float32)
    jstar = 3
    k[:, :, jstar, 0] = 20.0                                   # logit 8*20/sqrt(16) = 40
    G, I = oracle.score(synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k), 0, M, ts, True)
    assert abs(G[0, jstar] - N) < 1e-6 and abs(I[0, jstar] - 1.0) < 1e-6
    others = np.delete(np.arange(M), jstar)
    assert (G[0, others] < 1e-15).all() and (I[0, others] < 1e-15).all()
    assert (G[0, others] > 0).all()


def test_rank_one_logits_by_hand():
    """q_i = a_i e_0, k_l = b_l e_0: z = scale a_i b_l, softmax written out with math.exp."""
    a = [0.5, -1.0, 2.0]
    b = [1.0, -0.5, 0.25, 2.0, -2.0, 0.75]         # 3 vision keys then 3 text keys (bf16-exact)
    H, N, M, D = 1, 3, 3, 4
    q = np.zeros((1, H, N, D), np.float32)
    k = np.zeros((1, H, M + N, D), np.float32)
    q[0, 0, :, 0] = a
    k[0, 0, :, 0] = b
    G, I, A = oracle.score(synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k), 0, M, M, True, return_a=True)
    scale = 1.0 / math.sqrt(D)
    exp_a = np.zeros((N, M))
    for i in range(N):
        vis = range(M + i + 1)
        den = sum(math.exp(scale * a[i] * b[l]) for l in vis)
        for j in range(M):
            exp_a[i, j] = math.exp(scale * a[i] * b[j]) / den
    assert np.allclose(A[0], exp_a, rtol=1e-12)
    assert np.allclose(G[0], exp_a.sum(0), rtol=1e-6) and np.allclose(I[0], exp_a.max(0), rtol=1e-6)


def test_heads_are_averaged_before_the_max():
    """Two heads peaking on different text rows: max of the mean differs from mean of the max."""
    H, N, M, D = 2, 2, 2, 4
    q = np.zeros((1, H, N, D), np.float32)
    k = np.zeros((1, H, M + N, D), np.float32)
    q[0, 0, 0, 0] = 4.0   # head 0: text row 0 looks at vision key 0
    q[0, 1, 1, 0] = 4.0   # head 1: text row 1 looks at vision key 0
    k[0, :, 0, 0] = 4.0
    G, I, A = oracle.score(synth.f32_to_bf16_bits(q), synth.f32_to_bf16_bits(k), 0, M, M, True, return_a=True)
    p = oracle.attention(synth.f32_to_bf16_bits(q)[0], synth.f32_to_bf16_bits(k)[0], M, True)
    mean_then_max = p[:, :, :M].mean(0).max(0)
    max_then_mean = p[:, :, :M].max(1).mean(0)
    assert not np.allclose(mean_then_max, max_then_mean, rtol=1e-2)
    assert np.allclose(I[0], mean_then_max, rtol=1e-6)


@pytest.mark.parametrize("causal", [True, False])
def test_inequalities(causal):
    q, k, vs, M, ts, L = _rand_case(11, H=4, N=9, M=20)
    N = q.shape[2]
    G, I = oracle.score(q, k, vs, M, ts, causal)
    G, I = G.astype(np.float64), I.astype(np.float64)
    assert (I > 0).all() and (I <= G * (1 + 1e-6)).all() and (G <= N * I * (1 + 1e-6)).all()
    assert G.sum() <= N
    p = oracle.attention(q[0], k[0], ts, causal)
    mass_vis = p[:, :, vs:vs + M].mean(0).sum()
    mass_rest = p.mean(0).sum() - mass_vis
    assert abs(G.sum() - mass_vis) < 1e-5 and abs(mass_vis + mass_rest - N) < 1e-9


def test_equivariances():
    q, k, vs, M, ts, L = _rand_case(13, H=3, N=6, M=10, vis_start=0)
    G, I = oracle.score(q, k, vs, M, ts, True)
    rng = np.random.default_rng(0)
    perm = rng.permutation(M)
    k2 = k.copy()
    k2[:, :, :M] = k[:, :, perm]
    G2, I2 = oracle.score(q, k2, vs, M, ts, True)
    assert np.array_equal(G2[0], G[0][perm]) and np.array_equal(I2[0], I[0][perm])
    hp = rng.permutation(q.shape[1])
    G3, I3 = oracle.score(q[:, hp], k[:, hp], vs, M, ts, True)
    assert np.allclose(G3, G, rtol=1e-6) and np.allclose(I3, I, rtol=1e-6)
    # full mask: the order of the text queries does not matter
    Gf, If = oracle.score(q, k, vs, M, ts, False)
    tp = rng.permutation(q.shape[2])
    Gp, Ip = oracle.score(q[:, :, tp], k, vs, M, ts, False)
    assert np.allclose(Gp, Gf, rtol=1e-6) and np.allclose(Ip, If, rtol=1e-6)


def test_batch_entries_are_independent():
    w = synth.WORKLOADS["c1_tiny"].with_(batch=2, n_vis=24, n_txt=5, n_heads=2, hidden=256,
                                         n_salient=2, key_cnt=3, budget=8)
    d = synth.make_batch(w, with_values=False)
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    G1, I1 = oracle.score(d["q_text"][1:], d["k"][1:], w.vis_start, w.n_vis, w.txt_start)
    assert np.array_equal(G[1:], G1) and np.array_equal(I[1:], I1)


def test_planted_salient_keys_score_high():
    """The workload's planted keys (aligned with the mean text query) stand out in G."""
    w = synth.WORKLOADS["c1_tiny"].with_(n_vis=96, n_txt=16, n_heads=4, hidden=512, n_salient=4)
    d = synth.make_batch(w, with_values=False)
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    sal = d["salient_idx"][0]
    rest = np.setdiff1d(np.arange(w.n_vis), sal)
    assert G[0, sal].min() > np.median(G[0, rest]) * 1.5


# ---- the per-head reading of Eq. 10 --------------------------------------------------------------

def test_per_head_reading_coincides_with_one_head_and_dominates_otherwise():
    w = synth.WORKLOADS["c1_tiny"].with_(batch=2, n_vis=40, n_txt=6, n_heads=1, hidden=128, n_salient=2, key_cnt=0, budget=8)
    d = synth.make_batch(w, with_values=False)
    G1, I1 = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    G2, I2 = oracle.score_per_head(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    assert np.array_equal(G1, G2) and np.array_equal(I1, I2)            # H = 1: one reading
    w = w.with_(n_heads=4, hidden=512)
    d = synth.make_batch(w, with_values=False)
    G1, I1 = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    G2, I2 = oracle.score_per_head(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    assert np.allclose(G1, G2, rtol=1e-6)                                # G is linear in the heads
    assert np.all(I2 >= I1 * (1 - 1e-6)) and np.any(I2 > I1 * 1.01)      # a mean of maxima is at least the maximum of the mean
    # against the attention map itself: the definition written with numpy
    for b in range(w.batch):
        p = oracle.attention(d["q_text"][b], d["k"][b], w.txt_start)     # [H, N, L]
        pv = p[:, :, w.vis_start:w.vis_start + w.n_vis]
        assert np.allclose(I2[b], pv.max(axis=1).mean(axis=0), rtol=1e-6)
        assert np.allclose(G2[b], pv.mean(axis=0).sum(axis=0), rtol=1e-6)

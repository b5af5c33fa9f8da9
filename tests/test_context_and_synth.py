"""Pins for the size accounting (Tables 1, 3, 6), invariants of the upstream/downstream
context functions, and determinism of the seeded input generator."""
import os

import numpy as np

from oracle import context
from paper_2411_10803_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def test_kv_cache_megabytes_match_the_printed_tables():
    # the paper's rows all sit at 0.525 MB per token (2*32*4096*2 B = 0.524288 MB exactly),
    # to the printed digit except the 2880-token row, which is 0.1 MB above it
    for tokens, mb, *_ in _rows("kv_cache_tables.txt"):
        tokens, mb = int(tokens), float(mb)
        assert abs(tokens * 0.525 - mb) <= 0.1 + 1e-9
        assert abs(context.kv_cache_mb(tokens) - mb) <= 0.0015 * mb + 0.05


def test_compression_ratios_match_the_printed_tables():
    for kept, total, pct, *_ in _rows("compression_ratios.txt"):
        assert abs(100.0 * (1 - int(kept) / int(total)) - float(pct)) <= 0.05 + 1e-9


def test_local_spatial_merge_invariants():
    rng = np.random.default_rng(0)
    g = 6
    x = rng.standard_normal((g * g, 8))
    m, slots = context.local_spatial_merge(x, g, 2, tau=0.8)
    assert m.shape[0] == g * g and np.array_equal(slots, np.arange(g * g))   # random tokens: nothing merges
    x[[0, 1, g, g + 1]] = x[0]                                              # one window of identical tokens
    m, slots = context.local_spatial_merge(x, g, 2, tau=0.999)
    assert m.shape[0] == g * g - 3 and slots[0] == 0 and np.allclose(m[0], x[0])
    assert 1 not in slots and g not in slots and g + 1 not in slots
    m_all, _ = context.local_spatial_merge(np.ones((g * g, 8)), g, 2, tau=0.5)
    assert m_all.shape[0] == (g // 2) ** 2


def test_key_set_picks_outliers():
    rng = np.random.default_rng(1)
    H, M, D = 4, 64, 16
    q = rng.standard_normal((H, D))
    k = 0.05 * rng.standard_normal((H, M, D))
    O, a = context.key_set(q, k)
    assert abs(a.sum() - 1) < 1e-12
    k[:, 10] = 3 * q / np.linalg.norm(q, axis=1, keepdims=True)
    O2, a2 = context.key_set(q, k)
    assert 10 in O2 and a2[10] == a2.max()


def test_cache_policy_keeps_only_the_last_layers_set_after_layer_two():
    kept = [np.arange(10), np.arange(10), np.arange(8), np.array([0, 2, 4, 6]), np.array([0, 4])]
    out = context.cache_policy(kept, 5)
    assert np.array_equal(out[0], np.arange(10)) and np.array_equal(out[1], np.arange(10))
    for l in (2, 3, 4):
        assert np.array_equal(out[l], [0, 4])
        assert set(out[l]).issubset(set(kept[l]))


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.140625, 0.0], np.float32)
    # 1 + 2^-8 is exactly half-way between 1 and 1 + 2^-7 -> ties to even (1.0);
    # 1 + 3*2^-8 is half-way between 1+2^-7 and 1+2^-6 -> ties to even (1 + 2^-6)
    b = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.015625 and back[3] == -2.5 and back[5] == 0.0
    import torch
    t = torch.randn(1000, dtype=torch.float32)
    ref = t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(synth.f32_to_bf16_bits(t.numpy()), ref)


def test_generator_is_deterministic_and_per_request():
    w = synth.WORKLOADS["c1_tiny"].with_(batch=3, n_vis=32, n_txt=4, n_heads=2, hidden=256, n_salient=2,
                                         key_cnt=4, budget=8)
    a, b = synth.make_batch(w), synth.make_batch(w)
    for name in a:
        assert np.array_equal(a[name], b[name])
    one = synth.make_request(w, 2)
    assert np.array_equal(one["k"], a["k"][2]) and np.array_equal(one["hidden"], a["hidden"][2])
    lite = synth.make_request(w, 2, with_values=False)
    assert np.array_equal(lite["key_idx"], one["key_idx"]) and np.array_equal(lite["k"], one["k"])
    assert a["k"].shape == (3, 2, 36, 128) and a["hidden"].shape == (3, 36, 256)
    assert not np.array_equal(a["k"][0], a["k"][1])
    assert synth.sha256_of(a["k"]) == synth.sha256_of(b["k"])
    sub = synth.make_batch(w, requests=range(1, 3))
    assert np.array_equal(sub["k"], a["k"][1:3])


def test_video_workload_keys_are_correlated_across_frames():
    w = synth.WORKLOADS["c4_video"].with_(batch=1, n_vis=8 * 16, n_txt=4, n_heads=2, hidden=256, key_cnt=4, budget=8)
    d = synth.make_request(w, 0, with_values=False)
    k = synth.bf16_bits_to_f64(d["k"])[:, : w.n_vis].reshape(2, 8, 16, 128)
    c = np.mean([np.corrcoef(k[:, f].ravel(), k[:, f + 1].ravel())[0, 1] for f in range(7)])
    assert 0.85 < c < 0.95
    assert abs(k.std() - 1.0) < 0.05


def test_workload_table_shapes():
    w = synth.WORKLOADS
    assert w["c2_llava7b_b64"].seq_len == 640 and w["c3_next7b"].seq_len == 2944
    assert w["c4_video"].seq_len == 2144 and w["c5_13b_b64"].seq_len == 704 and w["c5_13b_b64"].hidden == 5120
    for x in w.values():
        assert x.hidden == x.n_heads * x.head_dim and x.key_cnt <= x.budget <= x.n_vis

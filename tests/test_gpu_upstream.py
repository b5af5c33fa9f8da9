"""GPU parity of the vision-encoding stage kernels (Local Spatial Merging, Key Retaining;
Sec. 3.3) against the numpy oracle of oracle/context.py.  Decisions that floating point takes
(merge a window or not, a token above the fence or not) are compared outside a narrow band
around the oracle's threshold; everything else is exact or within rounding."""
import numpy as np
import pytest
import torch

from oracle import context
from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import build as md_build
from paper_2411_10803_b200 import synth

from parity_util import bf16_bits, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    md_build.build()
    assert torch.cuda.is_available()


def _ulps_apart(a_bits, b_bits):
    """Distance of two bf16 bit patterns in units in the last place (same sign assumed or zero)."""
    a = a_bits.astype(np.int32)
    b = b_bits.astype(np.int32)
    a = np.where(a & 0x8000, 0x8000 - a, a)
    b = np.where(b & 0x8000, 0x8000 - b, b)
    return np.abs(a - b)


@pytest.mark.parametrize("B,grid,C,tau", [(3, 24, 1024, 0.8), (2, 8, 64, 0.5), (1, 64, 32, 0.8), (4, 6, 136, 0.9)])
def test_spatial_merge_matches_oracle(B, grid, C, tau):
    bits = synth.make_vit_tokens(77, B, grid, C, merge_frac=0.3)
    n = grid * grid
    merged = torch.zeros((B, n, C), dtype=torch.bfloat16, device="cuda")
    slots = torch.full((B, n), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros((B,), dtype=torch.int32, device="cuda")
    sims = torch.zeros((B, (grid // 2) ** 2), dtype=torch.float32, device="cuda")
    st = md.mustdrop_spatial_merge(B, grid, 2, C, tau, to_dev_bf16(bits), merged, slots, cnt, sims)
    assert st == md.MUSTDROP_OK
    torch.cuda.synchronize()
    got, got_slots, got_cnt, got_sims = bf16_bits(merged), slots.cpu().numpy(), cnt.cpu().numpy(), sims.cpu().numpy()
    x = synth.bf16_bits_to_f64(bits)
    n_merged = 0
    for b in range(B):
        ref_rows, ref_slots, ref_sims = context.local_spatial_merge(x[b], grid, 2, tau, return_sims=True)
        assert np.all(np.abs(ref_sims - tau) > 1e-3), "a window sits on the threshold: pick other data"
        assert np.allclose(got_sims[b], ref_sims, rtol=0, atol=2e-5)
        assert got_cnt[b] == len(ref_slots)
        assert np.array_equal(got_slots[b, :got_cnt[b]], ref_slots)
        gw = grid // 2
        for r, s in enumerate(ref_slots):
            y, xx = divmod(int(s), grid)
            was_merged = ref_sims[(y // 2) * gw + xx // 2] > tau
            if was_merged:
                n_merged += 1
                want = synth.f32_to_bf16_bits(ref_rows[r].astype(np.float32))
                assert _ulps_apart(got[b, r], want).max() <= 1        # one rounding of an fp32 average
            else:
                assert np.array_equal(got[b, r], bits[b, s])          # a copy
        assert not got[b, got_cnt[b]:].any()                          # later rows untouched
    assert n_merged > 0


def test_spatial_merge_extremes():
    B, grid, C = 2, 4, 64
    bits = synth.make_vit_tokens(5, B, grid, C, merge_frac=0.0)
    bits[1] = bits[1, :1]                                             # image 1: all tokens identical
    for tau, want in ((0.8, [16, 4]), (-2.0, [4, 4]), (2.0, [16, 16])):
        merged = torch.zeros((B, 16, C), dtype=torch.bfloat16, device="cuda")
        slots = torch.zeros((B, 16), dtype=torch.int32, device="cuda")
        cnt = torch.zeros((B,), dtype=torch.int32, device="cuda")
        assert md.mustdrop_spatial_merge(B, grid, 2, C, tau, to_dev_bf16(bits), merged, slots, cnt) == md.MUSTDROP_OK
        torch.cuda.synchronize()
        assert cnt.cpu().tolist() == want
        if want[1] == 4:      # identical tokens average to themselves, at the windows' first slots
            assert slots.cpu().numpy()[1, :4].tolist() == [0, 2, 8, 10]
            assert np.array_equal(bf16_bits(merged)[1, :4], bits[1, :4])


@pytest.mark.parametrize("B,H,D,M,n_out", [(3, 16, 64, 576, 20), (2, 4, 128, 100, 5), (1, 2, 8, 4096, 60), (2, 3, 256, 33, 2)])
def test_key_set_matches_oracle(B, H, D, M, n_out):
    qb, kb, planted = synth.make_cls_attention(31, B, H, D, M, n_out)
    key_max = 256
    a = torch.zeros((B, M), dtype=torch.float32, device="cuda")
    mu = torch.zeros((B,), dtype=torch.float32, device="cuda")
    ki = torch.full((B, key_max), -1, dtype=torch.int32, device="cuda")
    kc = torch.zeros((B,), dtype=torch.int32, device="cuda")
    assert md.mustdrop_key_set(B, H, D, M, key_max, to_dev_bf16(qb), to_dev_bf16(kb), a, mu, ki, kc) == md.MUSTDROP_OK
    torch.cuda.synchronize()
    q, k = synth.bf16_bits_to_f64(qb), synth.bf16_bits_to_f64(kb)
    for b in range(B):
        ref_o, ref_a = context.key_set(q[b], k[b])
        q1, q3 = np.quantile(ref_a, [0.25, 0.75])
        ref_mu = q3 + 1.5 * (q3 - q1)
        got_a = a.cpu().numpy()[b]
        assert np.allclose(got_a, ref_a, rtol=2e-3, atol=1e-10)
        assert abs(mu.cpu().numpy()[b] - ref_mu) <= 2e-3 * ref_mu
        got_o = ki.cpu().numpy()[b, :kc.cpu().numpy()[b]]
        assert np.all(np.diff(got_o) > 0)
        # identical sets, except for tokens within the tolerance band around the fence
        for j in np.setxor1d(got_o, ref_o):
            assert abs(ref_a[j] - ref_mu) <= 4e-3 * ref_mu, (b, j, ref_a[j], ref_mu)
        # the planted tokens are far above the fence on both sides
        if n_out * 4 < M and D >= 64:
            assert set(planted[b].tolist()) <= set(got_o.tolist())


def test_key_set_capacity_and_uniform_attention():
    B, H, D, M = 1, 2, 64, 64
    qb, kb, planted = synth.make_cls_attention(9, B, H, D, M, 10)
    ki = torch.full((B, 4), -1, dtype=torch.int32, device="cuda")
    kc = torch.zeros((B,), dtype=torch.int32, device="cuda")
    assert md.mustdrop_key_set(B, H, D, M, 4, to_dev_bf16(qb), to_dev_bf16(kb), None, None, ki, kc) == md.MUSTDROP_OK
    torch.cuda.synchronize()
    ref_o, ref_a = context.key_set(synth.bf16_bits_to_f64(qb)[0], synth.bf16_bits_to_f64(kb)[0])
    q1, q3 = np.quantile(ref_a, [0.25, 0.75])
    assert np.all(np.abs(ref_a - (q3 + 1.5 * (q3 - q1))) > 1e-2 * ref_a), "a token sits on the fence: pick other data"
    assert len(ref_o) > 4 and set(planted[0].tolist()) <= set(ref_o.tolist())
    assert kc.cpu().tolist() == [4] and ki.cpu().numpy()[0].tolist() == ref_o[:4].tolist()   # the lowest indices
    # identical keys: uniform attention 1/M, no token above the fence
    kb[:] = kb[:, :, :1]
    a = torch.zeros((B, M), dtype=torch.float32, device="cuda")
    assert md.mustdrop_key_set(B, H, D, M, 4, to_dev_bf16(qb), to_dev_bf16(kb), a, None, ki, kc) == md.MUSTDROP_OK
    torch.cuda.synchronize()
    assert kc.cpu().tolist() == [0]
    assert np.allclose(a.cpu().numpy(), 1.0 / M, rtol=1e-5)


def test_upstream_feeds_the_filter():
    """merge -> vis_cnt, key set -> key_idx, both consumed by a ragged filter layer on one stream."""
    w = synth.WORKLOADS["c1_tiny"].with_(batch=2, n_heads=2, hidden=256, n_txt=8, budget=64, key_cnt=0, n_salient=4)
    grid, C = 24, 128
    tok = synth.make_vit_tokens(3, w.batch, grid, C, merge_frac=0.4)
    merged = torch.zeros((w.batch, grid * grid, C), dtype=torch.bfloat16, device="cuda")
    slots = torch.zeros((w.batch, grid * grid), dtype=torch.int32, device="cuda")
    vis_cnt = torch.zeros((w.batch,), dtype=torch.int32, device="cuda")
    assert md.mustdrop_spatial_merge(w.batch, grid, 2, C, 0.8, to_dev_bf16(tok), merged, slots, vis_cnt) == md.MUSTDROP_OK
    qb, kb, _ = synth.make_cls_attention(4, w.batch, 4, 64, 200, 12)   # 200 < every merged count
    ki = torch.full((w.batch, 32), -1, dtype=torch.int32, device="cuda")
    kc = torch.zeros((w.batch,), dtype=torch.int32, device="cuda")
    assert md.mustdrop_key_set(w.batch, 4, 64, 200, 32, to_dev_bf16(qb), to_dev_bf16(kb), None, None, ki, kc) == md.MUSTDROP_OK
    d = synth.make_batch(w)
    f = md.Filter(md.config_for(w, key_max=32))
    q, k, v, hid = (to_dev_bf16(d[n]) for n in ("q_text", "k", "v", "hidden"))
    # the text rows must sit behind each request's own tokens: pack on the host with the counts
    torch.cuda.synchronize()
    cnt = vis_cnt.cpu().numpy()
    assert (cnt >= 200).all() and (cnt < 576).all()
    p = synth.pack_ragged(d, w, cnt)
    q, k, v, hid = (to_dev_bf16(p[n]) for n in ("q_text", "k", "v", "hidden"))
    f.filter_layer(q, k, v, hid, ki, kc, vis_cnt=vis_cnt)
    torch.cuda.synchronize()
    assert f.device_status() == (0, 0)
    kept, n_kept = f.kept_idx.cpu().numpy(), f.kept_cnt.cpu().numpy()
    for b in range(w.batch):
        assert n_kept[b] == 64 and kept[b].max() < cnt[b]
        assert set(ki.cpu().numpy()[b, :kc.cpu().numpy()[b]].tolist()) <= set(kept[b].tolist())
    f.close()

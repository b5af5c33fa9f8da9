"""Host-side checks of the C ABI: the library loads without a GPU, exports every declared
symbol, and rejects bad configurations synchronously."""
import os
import re

import pytest

from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import build as md_build
from paper_2411_10803_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    md_build.build()


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(mustdrop_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    L = md.lib()
    declared = _declared()
    assert {"mustdrop_filter_plan", "mustdrop_score", "mustdrop_select", "mustdrop_compact"} <= declared
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(md.EXPORTS) | (declared - set(md.EXPORTS))
    for name in md.EXPORTS:
        assert name in declared, name


def _cfg(**kw):
    w = synth.WORKLOADS["c1_tiny"]
    return md.config_for(w, **kw)


def test_valid_plan_and_workspace_size():
    st, plan, ws = md.mustdrop_filter_plan(_cfg())
    assert st == md.MUSTDROP_OK and plan and ws >= 256 and ws % 256 == 0
    assert md.mustdrop_plan_score_variant(plan) != "invalid plan"
    assert md.mustdrop_plan_destroy(plan) == md.MUSTDROP_OK
    assert md.mustdrop_status_string(md.MUSTDROP_ERR_BUDGET)


@pytest.mark.parametrize("kw,code", [
    (dict(batch=0), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(n_txt=0), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(vis_start=10), md.MUSTDROP_ERR_INVALID_ARG),            # vision span runs into the text span
    (dict(txt_start=500), md.MUSTDROP_ERR_INVALID_ARG),           # text before the end of the vision span
    (dict(seq_len=600), md.MUSTDROP_ERR_INVALID_ARG),             # text span leaves the sequence
    (dict(causal=2), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(mode=5), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(criteria=3), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(gamma=-1.0), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(alpha=float("nan")), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(scale=float("inf")), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(flags=8), md.MUSTDROP_ERR_INVALID_ARG),                 # unknown flag bit
    (dict(debug_score_variant=5), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(debug_score_variant=4, debug_cluster=33), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(debug_cluster=17), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(debug_filter_staged=2), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(debug_wait_cycles=-1), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(flags=1, seq_len=700), md.MUSTDROP_ERR_INVALID_ARG),    # rebuild needs the text directly behind the image
    (dict(k_stride_l=-8), md.MUSTDROP_ERR_INVALID_ARG),
    (dict(k_stride_l=64), md.MUSTDROP_ERR_INVALID_ARG),           # rows would overlap
    (dict(head_dim=64), md.MUSTDROP_ERR_UNSUPPORTED),
    (dict(n_txt=129, seq_len=576 + 129), md.MUSTDROP_ERR_UNSUPPORTED),
    (dict(n_vis=4097, txt_start=4097, seq_len=4097 + 32, budget=64), md.MUSTDROP_ERR_UNSUPPORTED),
    (dict(hidden=4100), md.MUSTDROP_ERR_UNSUPPORTED),
    (dict(k_stride_h=12), md.MUSTDROP_ERR_UNSUPPORTED),
    (dict(budget=0), md.MUSTDROP_ERR_BUDGET),
    (dict(budget=577), md.MUSTDROP_ERR_BUDGET),
    (dict(budget=8, key_max=16), md.MUSTDROP_ERR_BUDGET),
])
def test_bad_configurations_are_rejected(kw, code):
    st, plan, ws = md.mustdrop_filter_plan(_cfg(**kw))
    assert st == code and plan == 0 and ws == 0


def test_threshold_mode_needs_no_budget():
    st, plan, _ = md.mustdrop_filter_plan(_cfg(mode=md.MUSTDROP_MODE_THRESHOLD, budget=0))
    assert st == md.MUSTDROP_OK
    md.mustdrop_plan_destroy(plan)


def test_null_and_misaligned_arguments_launch_nothing():
    st, plan, _ = md.mustdrop_filter_plan(_cfg())
    assert st == md.MUSTDROP_OK
    try:
        assert md.lib().mustdrop_score(plan, None, None, None, None, None, None) == md.MUSTDROP_ERR_INVALID_ARG
        assert md.lib().mustdrop_score(plan, 256, 256, 256, 256, None, None) == md.MUSTDROP_ERR_WORKSPACE
        assert md.lib().mustdrop_score(plan, 256, 260, 256, 256, 256, None) == md.MUSTDROP_ERR_INVALID_ARG
        assert md.lib().mustdrop_select(plan, 256, 256, None, None, 256, 256, None, 256, None) == \
            md.MUSTDROP_ERR_INVALID_ARG                      # key_max > 0 needs key_idx / key_cnt
        assert md.lib().mustdrop_compact(plan, 256, 256, 256, None, None, None, None, None, None, None) == \
            md.MUSTDROP_ERR_INVALID_ARG                      # source without destination
        assert md.lib().mustdrop_compact(plan, 256, 256, None, None, None, None, None, None, None, None) == \
            md.MUSTDROP_OK                                   # nothing to do
        assert md.lib().mustdrop_score(0, 256, 256, 256, 256, 256, None) == md.MUSTDROP_ERR_INVALID_ARG
    finally:
        md.mustdrop_plan_destroy(plan)


def test_shard_ranges_partition_the_batch():
    from paper_2411_10803_b200.sharding import shard_range
    for batch in (0, 1, 7, 64):
        for world in (1, 2, 3, 8):
            spans = [shard_range(batch, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == batch
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def test_cache_compact_rejects_bad_sizes_without_a_gpu():
    ok = dict(n_layers=2, batch=2, n_heads=2, rows_in=40, vis_start=1, n_tail=4, ids_max=20, cap=10)
    for bad in (dict(n_layers=0), dict(cap=21), dict(rows_in=24), dict(n_tail=-1)):
        kw = dict(ok)
        kw.update(bad)
        assert md.mustdrop_cache_compact(256, 256, 256, 256, 256, 256, 256, 256, None, stream=0, **kw) == \
            md.MUSTDROP_ERR_INVALID_ARG
    assert md.mustdrop_cache_compact(256, 256, 256, 256, 256, 256, 256, 256, None, stream=0, head_dim=64, **ok) == \
        md.MUSTDROP_ERR_UNSUPPORTED
    assert md.mustdrop_cache_compact(256, 256, None, 256, 256, 256, 256, 256, None, stream=0, **ok) == \
        md.MUSTDROP_ERR_INVALID_ARG                                   # no layer_ids
    assert md.mustdrop_cache_compact(256, None, 256, 256, 256, 256, 256, 256, None, stream=0, **ok) == \
        md.MUSTDROP_ERR_INVALID_ARG                                   # v_out without v_cache
    assert md.mustdrop_cache_compact(264, 256, 256, 256, 256, 256, 256, 256, None, stream=0, **ok) == \
        md.MUSTDROP_ERR_INVALID_ARG                                   # misaligned


def test_upstream_calls_reject_bad_sizes_without_a_gpu():
    assert md.mustdrop_spatial_merge(1, 24, 3, 1024, 0.8, 256, 256, 256, 256, None, stream=0) == md.MUSTDROP_ERR_UNSUPPORTED
    assert md.mustdrop_spatial_merge(1, 25, 2, 1024, 0.8, 256, 256, 256, 256, None, stream=0) == md.MUSTDROP_ERR_UNSUPPORTED
    assert md.mustdrop_spatial_merge(1, 24, 2, 1020, 0.8, 256, 256, 256, 256, None, stream=0) == md.MUSTDROP_ERR_UNSUPPORTED
    assert md.mustdrop_spatial_merge(0, 24, 2, 1024, 0.8, 256, 256, 256, 256, None, stream=0) == md.MUSTDROP_ERR_INVALID_ARG
    assert md.mustdrop_spatial_merge(1, 24, 2, 1024, 0.8, None, 256, 256, 256, None, stream=0) == md.MUSTDROP_ERR_INVALID_ARG
    assert md.mustdrop_key_set(1, 16, 60, 576, 64, 256, 256, None, None, 256, 256, stream=0) == md.MUSTDROP_ERR_UNSUPPORTED
    assert md.mustdrop_key_set(1, 16, 64, 5000, 64, 256, 256, None, None, 256, 256, stream=0) == md.MUSTDROP_ERR_UNSUPPORTED
    assert md.mustdrop_key_set(1, 16, 64, 576, 0, 256, 256, None, None, 256, 256, stream=0) == md.MUSTDROP_ERR_INVALID_ARG
    assert md.mustdrop_key_set(1, 16, 64, 576, 64, 256, 264, None, None, 256, 256, stream=0) == md.MUSTDROP_ERR_INVALID_ARG


def test_plan_description_names_the_geometry_without_a_gpu():
    # no device: the planner assumes 148 SMs and clusters of at most 8 CTAs
    st, plan, _ = md.mustdrop_filter_plan(md.config_for(synth.WORKLOADS["c2_llava7b_b64"]))
    assert st == md.MUSTDROP_OK
    text = md.mustdrop_plan_describe(plan)
    assert "cluster 2" in text and "320 keys per CTA" in text and "filter = 1 launch" in text
    assert md.mustdrop_plan_filter_launches(plan) == 1
    md.mustdrop_plan_destroy(plan)
    st, plan, _ = md.mustdrop_filter_plan(md.config_for(synth.WORKLOADS["c2_llava7b_b64"],
                                                        flags=md.MUSTDROP_FLAG_PER_HEAD_MAX))
    # the per-head reading of Eq. 10 runs on the same one-launch kernel
    assert st == md.MUSTDROP_OK and md.mustdrop_plan_score_variant(plan) == "fused_cluster_tcgen05"
    assert md.mustdrop_plan_filter_launches(plan) == 1
    md.mustdrop_plan_destroy(plan)
    st, plan, _ = md.mustdrop_filter_plan(md.config_for(synth.WORKLOADS["c2_llava7b_b64"],
                                                        debug_score_variant=md.MUSTDROP_DEBUG_VARIANT_TWO_PASS))
    assert st == md.MUSTDROP_OK and md.mustdrop_plan_score_variant(plan) == "two_pass_mma"
    assert md.mustdrop_plan_filter_launches(plan) == 4
    md.mustdrop_plan_destroy(plan)
    assert md.mustdrop_plan_describe(0) == "" or md.mustdrop_plan_filter_launches(0) == -1


def test_filter_layer_rejects_bad_arguments_without_a_gpu():
    w = synth.WORKLOADS["c1_tiny"]
    st, plan, _ = md.mustdrop_filter_plan(md.config_for(w))
    assert st == md.MUSTDROP_OK
    good = dict(q_text=256, k=256, v=256, hidden=256, key_idx=256, key_cnt=256, g_out=256, i_out=256,
                kept_idx=256, kept_cnt=256, hidden_out=256, k_out=256, v_out=256)

    def call(workspace=256, **kw):
        a = dict(good)
        a.update(kw)
        return md.mustdrop_filter_layer(plan, workspace, 0, **a)

    assert call(q_text=None) == md.MUSTDROP_ERR_INVALID_ARG
    assert call(kept_cnt=None) == md.MUSTDROP_ERR_INVALID_ARG
    assert call(key_idx=None) == md.MUSTDROP_ERR_INVALID_ARG              # the plan has a key set
    assert call(hidden_out=None) == md.MUSTDROP_ERR_INVALID_ARG           # source without destination
    assert call(key_idx_out=256) == md.MUSTDROP_ERR_INVALID_ARG           # key_cnt_out missing
    assert call(vis_cnt=264) == md.MUSTDROP_ERR_INVALID_ARG               # misaligned
    assert call(workspace=None) == md.MUSTDROP_ERR_WORKSPACE
    md.mustdrop_plan_destroy(plan)
    # a ragged batch needs the text directly behind the image
    st, plan, _ = md.mustdrop_filter_plan(md.config_for(w, txt_start=w.txt_start + 8, seq_len=w.seq_len + 8))
    assert st == md.MUSTDROP_OK
    assert md.mustdrop_filter_layer(plan, 256, 0, vis_cnt=256, **good) == md.MUSTDROP_ERR_INVALID_ARG
    md.mustdrop_plan_destroy(plan)
    import pytest as _pytest
    with _pytest.raises(TypeError):
        md.mustdrop_filter_layer(0, 256, 0, no_such_field=1)

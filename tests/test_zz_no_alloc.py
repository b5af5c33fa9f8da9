"""mustdrop_score_static: the score call for callers that cannot allocate device memory
(an engine whose pool owns the device heap, a plug-in that must not touch its host's
allocator).  Its scratch is a fixed array inside the library, so it takes no workspace; its
results must equal those of mustdrop_score, and both must agree with the CPU oracle.  Checked
on two calls in a row, because every call reuses the same array and must not depend on what
the previous call left there; the device's free memory must read the same before and after
the second call (the first one may still load the library's code onto the device).

Collected last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2411_10803_b200 import binding as md
from paper_2411_10803_b200 import build as md_build
from paper_2411_10803_b200 import synth

from parity_util import SCORE_ATOL, SCORE_RTOL, to_dev_bf16


def _close(a, b):
    a, b = a.cpu().numpy().astype(np.float64), b.cpu().numpy().astype(np.float64)
    return bool(np.all(np.abs(a - b) <= SCORE_RTOL * np.abs(b) + SCORE_ATOL))


@pytest.mark.gpu
def test_static_scratch_score_matches_the_workspace_call_twice_in_a_row():
    md_build.build()
    shapes = [
        synth.WORKLOADS["c1_tiny"],
        synth.WORKLOADS["c1_tiny"].with_(batch=3, n_vis=333, n_txt=21, n_heads=3, hidden=384, key_cnt=4, budget=16),
    ]
    for call, w in enumerate(shapes):           # the second call runs over the first call's leftovers
        d = synth.make_batch(w, with_values=False)
        q, k = to_dev_bf16(d["q_text"]), to_dev_bf16(d["k"])
        f = md.Filter(md.config_for(w))
        g_ref, i_ref = f.score(q, k)
        g = torch.full_like(g_ref, float("nan"))
        i = torch.full_like(i_ref, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        st = md.mustdrop_score_static(f.plan, q, k, g, i)
        assert st == md.MUSTDROP_OK, md.mustdrop_status_string(st)
        torch.cuda.synchronize()
        free_after = torch.cuda.mem_get_info()[0]
        if call > 0:
            assert free_after == free_before, "the call changed the device's free memory"
        assert _close(g, g_ref) and _close(i, i_ref), "call %d differs from mustdrop_score" % call
        G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
        assert _close(g, torch.from_numpy(G)) and _close(i, torch.from_numpy(I)), "call %d differs from the oracle" % call
        f.close()


def test_static_scratch_score_refuses_plans_beyond_its_array():
    md_build.build()
    limit = md.mustdrop_score_static_max_rows()
    assert limit == 512 * 1024
    w = synth.WORKLOADS["c5_13b_b64"].with_(batch=128)          # 128 * 40 * 128 rows > limit
    assert w.batch * w.n_heads * w.n_txt > limit
    st, plan, _ = md.mustdrop_filter_plan(md.config_for(w))
    assert st == md.MUSTDROP_OK
    try:
        assert md.lib().mustdrop_score_static(plan, 256, 256, 256, 256, None) == md.MUSTDROP_ERR_SCRATCH_LIMIT
        assert "524288" in md.mustdrop_status_string(md.MUSTDROP_ERR_SCRATCH_LIMIT)
        assert md.lib().mustdrop_score_static(plan, 256, 260, 256, 256, None) == md.MUSTDROP_ERR_INVALID_ARG
    finally:
        md.mustdrop_plan_destroy(plan)

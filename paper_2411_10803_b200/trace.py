"""Per-head timeline of the fused score kernel (a diagnostic, not part of the filter).

Compiles the library once more with -DMUSTDROP_TRACE into a temporary directory: that build
writes a global-timer stamp per (CTA, head, pipeline event) into the workspace behind its
first 4096 bytes.  Runs the score call on a synthetic workload and prints, for a few CTAs, when
each stage of each head happened and the mean duration of the stages.

    python -m paper_2411_10803_b200.trace [workload]        # default c2_llava7b_b16
    python -m paper_2411_10803_b200.trace [workload] score|filter [stamps.npy]
    python -m paper_2411_10803_b200.trace [workload] filter # the one-launch filter call: also the
                                                            # CTA-level stamps (entry, prologue,
                                                            # scores stored, selection, gather)
"""
from __future__ import annotations

import ctypes
import glob
import os
import subprocess
import sys
import tempfile

import numpy as np

from . import binding as md
from . import build as md_build
from . import synth

EVENTS = ["tma_issue", "mma_full", "mma_tempty", "exp_start", "exp_done", "add_sfull", "add_eready", "add_done"]
CTA_EVENTS = ["entry", "prologue_done", "scores_stored", "score_part_left", "selection_done", "gather_done"]   # slots 8.. of head 0


def build_trace_library(out_dir: str) -> str:
    so = os.path.join(out_dir, "libmustdrop_trace.so")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + md_build.NVCC_FLAGS + ["-DMUSTDROP_TRACE", "-I", os.path.join(md_build.ROOT, "include"), "-I",
                                           md_build.CSRC, "-o", so] + md_build.sources() + ["-lcuda"]
    subprocess.check_call(cmd)
    return so


def main(argv) -> int:
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("the trace needs a CUDA device")
    w = synth.WORKLOADS[argv[1] if len(argv) > 1 else "c2_llava7b_b16"]
    whole = len(argv) > 2 and argv[2] == "filter"
    with tempfile.TemporaryDirectory() as tmp:
        L = ctypes.CDLL(build_trace_library(tmp))
        vp = ctypes.c_void_p
        L.mustdrop_filter_plan.argtypes = [ctypes.c_void_p, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
        L.mustdrop_score.argtypes = [vp] * 7
        L.mustdrop_filter.argtypes = [vp] * 17
        L.mustdrop_plan_describe.argtypes = [vp, ctypes.c_char_p, ctypes.c_size_t]
        host = synth.make_batch(w, with_values=whole)
        q = torch.from_numpy(host["q_text"].view(np.int16)).cuda()
        k = torch.from_numpy(host["k"].view(np.int16)).cuda()
        g = torch.empty((w.batch, w.n_vis), dtype=torch.float32, device="cuda")
        i = torch.empty_like(g)
        cfg = md.config_for(w).to_c()
        plan, ws_bytes = vp(), ctypes.c_size_t()
        if L.mustdrop_filter_plan(ctypes.byref(cfg), ctypes.byref(plan), ctypes.byref(ws_bytes)) != 0:
            raise RuntimeError("plan refused")
        text = ctypes.create_string_buffer(256)
        L.mustdrop_plan_describe(plan, text, 256)
        print(text.value.decode())
        n_cta = w.batch * 32
        ws = torch.zeros(max(int(ws_bytes.value), 4096 + n_cta * w.n_heads * 16 * 8), dtype=torch.uint8, device="cuda")
        stream = torch.cuda.current_stream().cuda_stream
        if whole:
            v = torch.from_numpy(host["v"].view(np.int16)).cuda()
            hid = torch.from_numpy(host["hidden"].view(np.int16)).cuda()
            ki, kc = torch.from_numpy(host["key_idx"]).cuda(), torch.from_numpy(host["key_cnt"]).cuda()
            kept = torch.zeros((w.batch, w.budget), dtype=torch.int32, device="cuda")
            cnt = torch.zeros((w.batch,), dtype=torch.int32, device="cuda")
            ho = torch.zeros((w.batch, w.budget, w.hidden), dtype=torch.int16, device="cuda")
            ko = torch.zeros((w.batch, w.n_heads, w.budget, 128), dtype=torch.int16, device="cuda")
            vo = torch.zeros_like(ko)
        for _ in range(3):
            if whole:
                st = L.mustdrop_filter(plan, q.data_ptr(), k.data_ptr(), v.data_ptr(), hid.data_ptr(),
                                       ki.data_ptr() if w.key_cnt else None, kc.data_ptr() if w.key_cnt else None,
                                       g.data_ptr(), i.data_ptr(), None, kept.data_ptr(), cnt.data_ptr(), ho.data_ptr(),
                                       ko.data_ptr(), vo.data_ptr(), ws.data_ptr(), stream)
            else:
                st = L.mustdrop_score(plan, q.data_ptr(), k.data_ptr(), g.data_ptr(), i.data_ptr(), ws.data_ptr(), stream)
            if st != 0:
                raise RuntimeError("call refused: %d" % st)
            torch.cuda.synchronize()
        t = ws[4096:4096 + n_cta * w.n_heads * 16 * 8].cpu().numpy().view(np.uint64).reshape(n_cta, w.n_heads, 16).astype(np.float64)
    if len(argv) > 3:   # third argument: keep the raw stamps (ns; [CTA][head][event]) for a closer look
        np.save(argv[3], t)
    used = [c for c in range(n_cta) if t[c, 0, 0] > 0]
    if not used:
        print("no stamps: the plan does not use the fused kernel")
        return 1
    print("CTAs with stamps:", len(used), "(stamps of even heads only where the exp warps alternate heads)")
    # CTA-level phases, relative to the earliest kernel entry of the grid
    entry0 = min(t[c, 0, 8] for c in used)
    names = CTA_EVENTS if whole else CTA_EVENTS[:4]
    rel = np.array([[(t[c, 0, 8 + e] - entry0) / 1e3 for e in range(len(names))] for c in used])
    first_tma = np.array([(t[c, 0, 0] - entry0) / 1e3 for c in used])
    first_full = np.array([(t[c, 0, 1] - entry0) / 1e3 for c in used])
    last_add = np.array([(t[c, (w.n_heads - 1) // 2 * 2, 7] - entry0) / 1e3 for c in used])
    print("phases (us after the first CTA's entry; min / median / max over CTAs):")
    for n, col in [(names[0], rel[:, 0]), (names[1], rel[:, 1]), ("first_tma_issue", first_tma), ("first_stage_full", first_full),
                   ("last_even_head_added", last_add)] + [(names[e], rel[:, e]) for e in range(2, len(names))]:
        col = col[col > -1e6]
        print("  %-22s %8.2f %8.2f %8.2f" % (n, col.min(), np.median(col), col.max()))
    for c in used[:2] + used[-1:]:
        t0 = t[c, 0, 0]
        print("CTA", c)
        for h in sorted({0, 2, 4, w.n_heads // 2 // 2 * 2, (w.n_heads - 1) // 2 * 2}):
            print("  head %02d " % h + " ".join("%s=%.2f" % (n, (t[c, h, e] - t0) / 1e3) for e, n in enumerate(EVENTS))
                  + (" landed=%.2f" % ((t[c, h, 14] - t0) / 1e3) if t[c, h, 14] > 0 else ""))
        done = t[c, :, 7]
        print("  add_done per head: mean %.2f us" % (np.diff(done)[4:].mean() / 1e3))
        if t[c, 4, 14] > 0:   # whole-stage plans: an onlooker stamps the landing of every stage
            hs = t[c, 4:]
            print("  stage: copies issued -> landed %.2f us, landed -> MMA thread takes it %.2f us, issue -> next issue "
                  "into the same stage %.2f us" % ((hs[:, 14] - hs[:, 0]).mean() / 1e3, (hs[:, 2] - hs[:, 14]).mean() / 1e3,
                                                  np.diff(t[c, 4:, 0]).mean() / 1e3))
        ev = t[c, 4::2]
        print("  exp stage %.2f us, exp_done -> statistics complete %.2f us, add stage %.2f us" % (
            (ev[:, 4] - ev[:, 3]).mean() / 1e3, (ev[:, 5] - ev[:, 4]).mean() / 1e3, (ev[:, 7] - ev[:, 6]).mean() / 1e3))
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))

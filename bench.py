#!/usr/bin/env python
"""Benchmark of the vision-token filter: one step = score + select + compact over one batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints one JSON line (rank 0).  `value` is vision tokens filtered per second with the inputs
resident in device memory; `e2e` is the same metric with pinned host inputs copied in and
results copied out every step; `roofline` describes the dominant kernel (the score call)
against the measured HBM copy bandwidth; `cpu_baseline` is the CPU oracle on a bounded sample.
With N > 1 (torchrun) every rank filters its own batch: requests are independent, so there
is no collective on the data path (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2411_10803_b200 import synth  # noqa: E402

METRIC = "vision tokens filtered/sec (score+select+compact)"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "c2_llava7b_b64"
FALLBACK_HBM_GBS = 6650.0


# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, from the ncu
# captures summarised under profiles/.  Keyed by (workload, budget, "filter" | "score", kernel
# variant); anything else (or a kernel changed since its capture) reports null.
NCU_TRAFFIC_BYTES = {
    ("c2_llava7b_b64", 64, "filter", "fused_cluster_tcgen05"): 468290816 + 43839488,   # profiles/filter_kernel_c2_llava7b_b64.md
    ("c2_llava7b_b64", 64, "score", "fused_cluster_tcgen05"): 369175040 + 2975232,     # profiles/score_fused_kernel_c2_llava7b_b64.md
}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def bytes_model(w):
    """Algorithmic bytes per step (whole batch)."""
    B, H, D, L, N, M, Kp = w.batch, w.n_heads, w.head_dim, w.seq_len, w.n_txt, w.n_vis, w.budget
    k_bytes = B * H * L * D * 2
    q_bytes = B * H * N * D * 2
    out_bytes = B * Kp * (w.hidden + 2 * H * D) * 2
    score_bytes = k_bytes + q_bytes + 2 * B * M * 4
    return {
        "score": score_bytes,                      # K + Q_text read, G and I written
        "headline": k_bytes + q_bytes + out_bytes,  # K + Q_text + compacted outputs
        "full": k_bytes + q_bytes + 2 * out_bytes,  # + the gather's source rows
        "h2d": k_bytes * 2 + q_bytes + B * L * w.hidden * 2 + B * (max(w.key_cnt, 1) + 1) * 4,
        "d2h": out_bytes + B * (Kp + 1) * 4,
    }


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while the GPU is busy."""

    def __init__(self, device_index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            handle = None
            try:
                import torch
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                handle = None
            if handle is None:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = device_index
                if vis:
                    try:
                        idx = int(vis.split(",")[device_index])
                    except Exception:
                        idx = device_index
                handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.h = handle
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._halt.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_step(w, requests):
    """The CPU oracle over the given requests: score + select + compact.  Returns seconds."""
    import oracle
    d = synth.make_batch(w, requests=requests)
    t0 = time.perf_counter()
    G, I = oracle.score(d["q_text"], d["k"], w.vis_start, w.n_vis, w.txt_start)
    kidx = d["key_idx"] if w.key_cnt else None
    kcnt = d["key_cnt"] if w.key_cnt else None
    kept, cnt, _, _ = oracle.select(G, I, w.seq_len, kidx, kcnt, budget=w.budget)
    oracle.compact(kept, cnt, w.vis_start, d["hidden"], d["k"], d["v"])
    return time.perf_counter() - t0


def run_reference(args, w):
    """The oracle as it stands, timed on the host cores: each step is a bounded sample of requests."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    probe = oracle_step(w, range(0, 1))                                 # also warms the page cache
    budget_s = 150.0
    per_step = int(max(1, min(8, w.batch, budget_s / max(probe * (args.steps + args.warmup), 1e-9))))
    for i in range(args.warmup):
        oracle_step(w, range(0, per_step))
    total = 0.0
    for i in range(args.steps):
        lo = (i * per_step) % max(w.batch - per_step + 1, 1)
        total += oracle_step(w, range(lo, lo + per_step))
    ms = 1e3 * total / max(args.steps, 1)
    value = per_step * w.n_vis / (ms / 1e3)
    sample = "%d of the %d requests per step (score+select+compact)" % (per_step, w.batch)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "n_vis": w.n_vis, "n_txt": w.n_txt, "n_heads": w.n_heads,
                   "hidden": w.hidden, "budget": w.budget, "key_set": w.key_cnt, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def quick_measure(torch, md, w, steps, dev):
    """Step time of the one-call filter on another workload (device-resident inputs, back-to-back steps)."""
    host = synth.make_batch(w)
    t = {n: torch.from_numpy(host[n].view(np.int16)).to(dev).view(torch.bfloat16) for n in ("q_text", "k", "v", "hidden")}
    ki, kc = (torch.from_numpy(host["key_idx"]).to(dev), torch.from_numpy(host["key_cnt"]).to(dev)) if w.key_cnt else (None, None)
    f = md.Filter(md.config_for(w), device=dev)
    stream = torch.cuda.current_stream()
    ms = _time_steps(torch, stream, lambda: f.filter(t["q_text"], t["k"], t["v"], t["hidden"], ki, kc, stream=stream), steps, 5)
    code, _ = f.device_status()
    plan = f.description
    f.close()
    if code != 0:
        raise RuntimeError("device status %d on %s" % (code, w.name))
    bm = bytes_model(w)
    peak, _ = measured_peak()
    return {"workload": w.name, "batch": w.batch, "budget": w.budget, "ms_per_step": ms,
            "tokens_per_s": w.batch * w.n_vis / (ms / 1e3), "headline_frac_of_peak": bm["headline"] / (ms / 1e3) / 1e9 / peak,
            "plan": plan}


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2411_10803_b200 import binding as md
    from paper_2411_10803_b200 import build as md_build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the filter has no CPU path")
    torch.cuda.set_device(local_rank)
    if rank == 0:
        md_build.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    dev = torch.device("cuda", local_rank)

    # every rank filters its own batch of w.batch requests (distinct request numbers per rank)
    reqs = range(rank * w.batch, (rank + 1) * w.batch)
    host = synth.make_batch(w, requests=reqs)

    def pinned(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else
                                np.ascontiguousarray(a)).pin_memory()

    h_q, h_k, h_v, h_hid = (pinned(host[n]) for n in ("q_text", "k", "v", "hidden"))
    h_ki, h_kc = pinned(host["key_idx"]), pinned(host["key_cnt"])
    d_q, d_k, d_v, d_hid = (t.to(dev).view(torch.bfloat16) for t in (h_q, h_k, h_v, h_hid))
    d_ki, d_kc = h_ki.to(dev), h_kc.to(dev)
    use_keys = w.key_cnt > 0
    f = md.Filter(md.config_for(w), device=dev)
    stream = torch.cuda.current_stream()

    ki, kc = (d_ki, d_kc) if use_keys else (None, None)
    single_call = args.path != "staged"     # the one-call entry point (one launch where the plan allows)

    def step():
        if single_call:
            f.filter(d_q, d_k, d_v, d_hid, ki, kc, stream=stream)
        else:
            f.score(d_q, d_k, stream)
            f.select(ki, kc, stream=stream, want_s=False)
            f.compact(d_hid, d_k, d_v, stream=stream)

    launches_per_step = f.filter_launches if single_call else {"two_pass_mma": 2}.get(f.score_variant, 1) + 2
    one_kernel = single_call and launches_per_step == 1

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler is not None:
        sampler.start()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    # timed region: exactly K steps between two events on the launching stream.  No events are
    # recorded inside it, so the kernels' programmatic dependent launches overlap as in real use.
    K = args.steps
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    host_t0 = time.perf_counter()
    for s in range(K):
        step()
    host_enqueue_ms = 1e3 * (time.perf_counter() - host_t0) / K   # host time to enqueue one step
    t_end.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    elapsed_ms = t_begin.elapsed_time(t_end)

    # per-call durations for the roofline: a second pass over the same K steps with an event
    # around every call (the events serialise the calls, so these add up to more than a step)
    f.score(d_q, d_k, stream)            # one untimed round: the separate kernels may not have run yet
    f.select(ki, kc, stream=stream, want_s=False)
    f.compact(d_hid, d_k, d_v, stream=stream)
    f.filter(d_q, d_k, d_v, d_hid, ki, kc, stream=stream)
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(K)]
    for s in range(K):
        ev[s][0].record(stream)
        f.score(d_q, d_k, stream)
        ev[s][1].record(stream)
        f.select(ki, kc, stream=stream, want_s=False)
        ev[s][2].record(stream)
        f.compact(d_hid, d_k, d_v, stream=stream)
        ev[s][3].record(stream)
        f.filter(d_q, d_k, d_v, d_hid, ki, kc, stream=stream)
        ev[s][4].record(stream)
    torch.cuda.synchronize()
    t_score = statistics.mean(ev[s][0].elapsed_time(ev[s][1]) for s in range(K))
    t_select = statistics.mean(ev[s][1].elapsed_time(ev[s][2]) for s in range(K))
    t_compact = statistics.mean(ev[s][2].elapsed_time(ev[s][3]) for s in range(K))
    t_filter = statistics.mean(ev[s][3].elapsed_time(ev[s][4]) for s in range(K))
    code, detail = f.device_status()
    if code != 0:
        raise RuntimeError("device status %d (detail %d) after the timed region" % (code, detail))

    # end to end: pinned host inputs in, results out, every step
    o_idx = torch.empty(f.kept_idx.shape, dtype=torch.int32).pin_memory()
    o_cnt = torch.empty(f.kept_cnt.shape, dtype=torch.int32).pin_memory()
    o_h = torch.empty(f.hidden_out.shape, dtype=torch.bfloat16).pin_memory()
    o_k = torch.empty(f.k_out.shape, dtype=torch.bfloat16).pin_memory()
    o_v = torch.empty(f.v_out.shape, dtype=torch.bfloat16).pin_memory()
    s_q, s_k, s_v, s_hid = (torch.empty_like(t) for t in (d_q, d_k, d_v, d_hid))
    s_ki, s_kc = torch.empty_like(d_ki), torch.empty_like(d_kc)

    def e2e_step():
        s_q.view(torch.int16).copy_(h_q, non_blocking=True)
        s_k.view(torch.int16).copy_(h_k, non_blocking=True)
        s_v.view(torch.int16).copy_(h_v, non_blocking=True)
        s_hid.view(torch.int16).copy_(h_hid, non_blocking=True)
        s_ki.copy_(h_ki, non_blocking=True)
        s_kc.copy_(h_kc, non_blocking=True)
        if single_call:
            f.filter(s_q, s_k, s_v, s_hid, s_ki if use_keys else None, s_kc if use_keys else None, stream=stream)
        else:
            f.score(s_q, s_k, stream)
            f.select(s_ki if use_keys else None, s_kc if use_keys else None, stream=stream, want_s=False)
            f.compact(s_hid, s_k, s_v, stream=stream)
        o_idx.copy_(f.kept_idx, non_blocking=True)
        o_cnt.copy_(f.kept_cnt, non_blocking=True)
        o_h.copy_(f.hidden_out, non_blocking=True)
        o_k.copy_(f.k_out, non_blocking=True)
        o_v.copy_(f.v_out, non_blocking=True)

    e2e_steps = max(3, min(K, 20))
    e2e_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    clocks = sampler.finish() if sampler is not None else None

    # max over ranks
    if world > 1:
        t = torch.tensor([elapsed_ms, e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms, e2e_ms = float(t[0]), float(t[1])
    ms_per_step = elapsed_ms / K
    tokens_per_step = world * w.batch * w.n_vis
    value = tokens_per_step / (ms_per_step / 1e3)
    e2e_value = tokens_per_step / (e2e_ms / 1e3)

    if rank == 0:
        bm = bytes_model(w)
        peak, peak_kind = measured_peak()
        # dominant kernel: the single-launch filter kernel (score + selection + gather: K, Q_text,
        # gathered rows read, compacted rows written), else the score kernel (K, Q_text read)
        if one_kernel:
            dom_name, dom_bytes, dom_ms = "filter (%s + select + gather tail)" % f.score_variant, bm["full"], t_filter
        else:
            dom_name, dom_bytes, dom_ms = "score (%s)" % f.score_variant, bm["score"], t_score
        achieved = dom_bytes / (dom_ms / 1e3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "n_vis": w.n_vis, "n_txt": w.n_txt,
                       "n_heads": w.n_heads, "hidden": w.hidden, "budget": w.budget, "key_set": w.key_cnt,
                       "parallelism": "dp%d (independent requests, no collective)" % world,
                       "l2": "inputs exceed L2 (K alone is %.0f MB per GPU)" % (bm["score"] / 1e6),
                       "score_variant": f.score_variant, "plan": f.description,
                       "path": ("mustdrop_filter, %d launch(es) per step" % launches_per_step) if single_call
                       else "mustdrop_score + mustdrop_select + mustdrop_compact"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": bm["h2d"], "d2h_bytes_per_step": bm["d2h"],
                    "ms_per_step": e2e_ms, "steps": e2e_steps},
            "gpu_launches": launches_per_step * K,
            "host_enqueue_ms_per_step": host_enqueue_ms,
            "kernel_ms": {"score": t_score, "select": t_select, "compact": t_compact, "filter_call": t_filter,
                          "how": "second pass over the same steps with an event around every call "
                                 "(the three separate calls, then the one-call filter)"},
            "hbm_headline": {"bytes_per_step": bm["headline"], "gbs": bm["headline"] / (ms_per_step / 1e3) / 1e9,
                             "frac_of_peak": bm["headline"] / (ms_per_step / 1e3) / 1e9 / peak, "peak_kind": peak_kind},
            "roofline": {"kernel": dom_name, "bound": "hbm", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_BYTES.get((w.name, w.budget, dom_name.split(" ")[0], f.score_variant)),
                         "peak_kind": peak_kind, "algorithmic_bytes": dom_bytes, "ms": dom_ms},
            "clocks": clocks,
        }
        if world == 1 and not args.no_sweep:
            # the other listed configurations, for the record (not the benchmark line's metric)
            also = []
            b16 = synth.WORKLOADS["c2_llava7b_b16"]
            for item in (b16.with_(budget=192), b16.with_(budget=128), b16.with_(budget=64),
                         synth.WORKLOADS["c3_next7b"], synth.WORKLOADS["c4_video"], synth.WORKLOADS["c5_13b_b64"]):
                if item.name != w.name or item.budget != w.budget:
                    also.append(quick_measure(torch, md, item, 50, dev))
            line["other_workloads"] = also
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            probe = oracle_step(w, range(0, 1))
            n_req = int(max(1, min(w.batch, 15.0 / max(probe, 1e-6))))
            secs = oracle_step(w, range(0, n_req))
            line["cpu_baseline"] = {"value": n_req * w.n_vis / secs, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": "%d of the %d requests, score+select+compact, %.1f s" % (n_req, w.batch, secs)}
        print(json.dumps(line), flush=True)
    f.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def _time_steps(torch, stream, fn, steps, warmup):
    for _ in range(max(warmup, 3)):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def run_layers(args, w):
    """Side measurement: a chain of pruning layers on a ragged batch (mustdrop_filter_layer),
    every layer feeding the next on one stream.  Prints its own JSON line (single GPU)."""
    import torch
    from paper_2411_10803_b200 import binding as md
    from paper_2411_10803_b200 import build as md_build
    md_build.build()
    torch.cuda.set_device(0)
    budgets = [int(x) for x in args.layer_budgets.split(",")]
    caps = [w.n_vis] + budgets[:-1]
    cnt = synth.draw_vis_cnt(w)
    cnts = [cnt]
    for kp in budgets[:-1]:
        cnts.append(np.minimum(cnts[-1], kp))
    filters, dev, moved = [], [], 0
    for l, (cap, kp) in enumerate(zip(caps, budgets)):
        wl = w.with_(n_vis=cap, budget=kp, seed=w.seed + 100 * l, key_cnt=w.key_cnt if l == 0 else 0,
                     n_salient=min(w.n_salient, cap))
        p = synth.pack_ragged(synth.make_batch(wl), wl, cnts[l])
        filters.append(md.Filter(md.config_for(wl, key_max=w.key_cnt, flags=md.MUSTDROP_FLAG_REBUILD_SEQUENCE)))
        dev.append([torch.from_numpy(p[n].view(np.int16)).cuda().view(torch.bfloat16)
                    for n in ("q_text", "k", "v", "hidden")])
        if l == 0:
            ki0, kc0 = torch.from_numpy(p["key_idx"]).cuda(), torch.from_numpy(p["key_cnt"]).cuda()
        row = (w.hidden + 2 * w.n_heads * w.head_dim) * 2
        for b in range(w.batch):
            lb = w.vis_start + int(cnts[l][b]) + w.n_txt
            out_rows = w.vis_start + min(int(cnts[l][b]), kp) + w.n_txt
            moved += w.n_heads * (lb + w.n_txt) * w.head_dim * 2 + 2 * out_rows * row   # K + Q read, rows read + written
    vc0 = torch.from_numpy(cnt).cuda()
    stream = torch.cuda.current_stream()

    def step():
        ki, kc, vc, orig = ki0, kc0, vc0, None
        for l, f in enumerate(filters):
            q, k, v, hid = dev[l]
            f.filter_layer(q, k, v, hid, ki if w.key_cnt else None, kc if w.key_cnt else None, vis_cnt=vc,
                           orig_idx=orig, stream=stream)
            ki, kc, vc, orig = f.key_idx_out, f.key_cnt_out, f.kept_cnt, f.orig_out

    ms = _time_steps(torch, stream, step, args.steps, args.warmup)
    for f in filters:
        code, detail = f.device_status()
        if code != 0:
            raise RuntimeError("device status %d (detail %d)" % (code, detail))
    peak, peak_kind = measured_peak()
    tokens = int(cnt.sum())
    print(json.dumps({
        "op": "layers", "metric": "vision tokens filtered/sec through %d pruning layers" % len(budgets),
        "value": tokens / (ms / 1e3), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "ms_per_step": ms,
        "config": {"workload": w.name + " ragged", "batch": w.batch, "vis_cnt_mean": float(cnt.mean()),
                   "capacities": caps, "budgets": budgets, "launches_per_step": sum(f.filter_launches for f in filters)},
        "roofline": {"bound": "hbm", "achieved": moved / (ms / 1e3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": moved / (ms / 1e3) / 1e9 / peak, "peak_kind": peak_kind, "algorithmic_bytes": moved,
                     "traffic": None},
        "data": "synthetic"}), flush=True)
    for f in filters:
        f.close()


def run_cache(args, w):
    """Side measurement: decoding-stage cache compaction of all sparse layers in one launch."""
    import torch
    from paper_2411_10803_b200 import binding as md
    from paper_2411_10803_b200 import build as md_build
    md_build.build()
    torch.cuda.set_device(0)
    Lyr, B, H, D = args.cache_layers, w.batch, w.n_heads, w.head_dim
    ids_max = cap = w.budget
    n_tail, vs = w.n_txt, w.vis_start
    rng = np.random.Generator(np.random.PCG64(w.seed + 5))
    few_cnt = rng.integers(int(0.6 * cap), int(0.8 * cap) + 1, B).astype(np.int32)      # 64 -> about 45 (Table 3)
    s_few = np.full((B, cap), -1, np.int32)
    layer_ids = np.full((Lyr, B, ids_max), -1, np.int32)
    layer_cnt = np.full((Lyr, B), ids_max, np.int32)
    for b in range(B):
        held = np.sort(rng.choice(w.n_vis, ids_max, replace=False))
        layer_ids[:, b] = held
        s_few[b, :few_cnt[b]] = np.sort(rng.choice(held, few_cnt[b], replace=False))
    R = vs + ids_max + n_tail
    kc = torch.randn((Lyr, B, H, R, D), device="cuda", dtype=torch.bfloat16)
    vc = torch.randn((Lyr, B, H, R, D), device="cuda", dtype=torch.bfloat16)
    ko = torch.zeros((Lyr, B, H, vs + cap + n_tail, D), device="cuda", dtype=torch.bfloat16)
    vo = torch.zeros_like(ko)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    args_dev = [torch.from_numpy(a).cuda() for a in (layer_ids, layer_cnt, s_few, few_cnt)]
    stream = torch.cuda.current_stream()

    def step():
        st = md.mustdrop_cache_compact(kc, vc, *args_dev, ko, vo, ws, stream, n_layers=Lyr, batch=B, n_heads=H,
                                       rows_in=R, vis_start=vs, n_tail=n_tail, ids_max=ids_max, cap=cap)
        if st != md.MUSTDROP_OK:
            raise RuntimeError("mustdrop_cache_compact: %d" % st)

    ms = _time_steps(torch, stream, step, args.steps, args.warmup)
    if ws[:4].cpu().numpy().view(np.int32)[0] != 0:
        raise RuntimeError("device status set")
    rows = int((vs + few_cnt + n_tail).sum())
    moved = 2 * 2 * Lyr * rows * H * D * 2     # K and V, read and written
    peak, peak_kind = measured_peak()
    print(json.dumps({
        "op": "cache_compact", "metric": "cache rows compacted/sec (K and V, all sparse layers)",
        "value": Lyr * rows / (ms / 1e3), "unit": "rows/s", "n_gpus": 1, "steps": args.steps, "ms_per_step": ms,
        "config": {"layers": Lyr, "batch": B, "n_heads": H, "held_per_layer": ids_max, "s_few_mean": float(few_cnt.mean()),
                   "tail_rows": n_tail},
        "roofline": {"bound": "hbm", "achieved": moved / (ms / 1e3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": moved / (ms / 1e3) / 1e9 / peak, "peak_kind": peak_kind, "algorithmic_bytes": moved,
                     "traffic": None},
        "data": "synthetic"}), flush=True)


def run_upstream(args, w):
    """Side measurement: the vision-encoding stage kernels (spatial merge, [CLS] key set)."""
    import torch
    from paper_2411_10803_b200 import binding as md
    from paper_2411_10803_b200 import build as md_build
    md_build.build()
    torch.cuda.set_device(0)
    B, grid, C, H, D = w.batch, 24, 1024, 16, 64          # CLIP ViT-L/14 at 336 px: 24 x 24 patches, 1024 channels
    M = grid * grid
    tok = torch.from_numpy(synth.make_vit_tokens(w.seed, B, grid, C).view(np.int16)).cuda().view(torch.bfloat16)
    qb, kb, _ = synth.make_cls_attention(w.seed, B, H, D, M, 29)
    q = torch.from_numpy(qb.view(np.int16)).cuda().view(torch.bfloat16)
    k = torch.from_numpy(kb.view(np.int16)).cuda().view(torch.bfloat16)
    merged = torch.zeros((B, M, C), dtype=torch.bfloat16, device="cuda")
    slots = torch.zeros((B, M), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((B,), dtype=torch.int32, device="cuda")
    ki = torch.zeros((B, 64), dtype=torch.int32, device="cuda")
    kc = torch.zeros((B,), dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    peak, peak_kind = measured_peak()

    def merge():
        st = md.mustdrop_spatial_merge(B, grid, 2, C, 0.8, tok, merged, slots, cnt, None, stream)
        assert st == md.MUSTDROP_OK

    def keys():
        st = md.mustdrop_key_set(B, H, D, M, 64, q, k, None, None, ki, kc, stream)
        assert st == md.MUSTDROP_OK

    ms_m = _time_steps(torch, stream, merge, args.steps, args.warmup)
    ms_k = _time_steps(torch, stream, keys, args.steps, args.warmup)
    kept = int(cnt.sum())
    bytes_m = B * M * C * 2 + kept * C * 2
    bytes_k = B * H * M * D * 2
    print(json.dumps({
        "op": "upstream", "unit": "images/s", "n_gpus": 1, "steps": args.steps,
        "config": {"batch": B, "grid": grid, "channels": C, "vit_heads": H, "vit_head_dim": D,
                   "tokens_after_merge_mean": kept / B, "key_set_mean": float(kc.float().mean())},
        "spatial_merge": {"ms": ms_m, "images_per_s": B / (ms_m / 1e3), "algorithmic_bytes": bytes_m,
                          "achieved_gbs": bytes_m / (ms_m / 1e3) / 1e9, "frac": bytes_m / (ms_m / 1e3) / 1e9 / peak},
        "key_set": {"ms": ms_k, "images_per_s": B / (ms_k / 1e3), "algorithmic_bytes": bytes_k,
                    "achieved_gbs": bytes_k / (ms_k / 1e3) / 1e9, "frac": bytes_k / (ms_k / 1e3) / 1e9 / peak},
        "peak": peak, "peak_kind": peak_kind, "data": "synthetic"}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--budget", type=int, default=0, help="override the workload's keep budget")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--path", default="filter", choices=["filter", "staged"],
                    help="filter: the one-call entry point; staged: score, select and compact as three calls")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the short runs of the other listed configurations")
    ap.add_argument("--op", default="filter", choices=["filter", "layers", "cache_compact", "upstream"],
                    help="filter: the benchmark proper; layers / cache_compact: side measurements (1 GPU)")
    ap.add_argument("--layer-budgets", default="192,128,64", help="--op layers: keep budget of each pruning layer")
    ap.add_argument("--cache-layers", type=int, default=30, help="--op cache_compact: layers that keep only S_few")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.budget:
        w = w.with_(budget=args.budget)
    if args.op == "layers":
        run_layers(args, w)
    elif args.op == "cache_compact":
        run_cache(args, w)
    elif args.op == "upstream":
        run_upstream(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

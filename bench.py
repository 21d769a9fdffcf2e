#!/usr/bin/env python
"""Benchmark of the VocabTrim hot path on B200.

Headline (the JSON line's `value`): microseconds per draft step of the trimmed drafter LM head on
the Llama-3.2-3B-class workload (V=128256, d=3072, K=32768, B=1, greedy + top-8 log-probs),
one `vt_draft_head` call per step, inputs resident in HBM, W_trim rotated over several copies so
that every step reads its weights from HBM and not from L2.

Also on the line: `e2e` (same step through `vt_draft_head_host`: pinned host inputs copied in and
results copied out every step), `roofline` (achieved HBM GB/s of the head kernel against the
measured copy bandwidth), `cpu_baseline` (the fp64 CPU oracle timed on a bounded sample), `clocks`
(SM clock and throttle reasons sampled during the timed region), `gpu_launches`, and, at N=1, the
sweep of K for the tree-drafting head, the full-vocabulary head and the corpus-scale vocabulary
build (Gtok/s).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the
same step on its own GPU; the path has no exchange step, so there is no collective in the data
path (only the barrier and the max-over-ranks of the timing).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import vt_inputs  # noqa: E402

V = vt_inputs.LLAMA3_VOCAB
HEAD = dict(d=3072, K=32768, B=1, topk=8, temp=1.0)            # config 2: chain drafting
TREE = dict(d=4096, B=10, topk=10, temp=0.7)                   # config 3: tree drafting
TREE_KS = (8192, 16384, 32768, 65536, V)
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0

PROFILE_KERNEL_SOURCES = {           # kernel -> the sources whose change invalidates its captured counters
    "k_head_stream": ("vt_head_skinny.cu", "vt_head_common.cuh"),
    "k_head_dense": ("vt_head_dense.cu", "vt_head_common.cuh"),
    "k_hist_packed": ("vt_hist.cu",),
}


def source_digest(kernel: str) -> str:
    """Short hash of the source files a kernel is built from (what a profile summary records)."""
    import hashlib

    h = hashlib.sha256()
    for name in PROFILE_KERNEL_SOURCES[kernel]:
        h.update(open(os.path.join(ROOT, "paper_2506_22694_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def profile_traffic(kernel: str, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` on `workload`, read from the
    ncu summary under profiles/ (a line `traffic_bytes_per_launch[<kernel>|<workload>] = <bytes> @ <digest>`).
    None when no capture exists or the kernel's sources changed since it was taken."""
    import glob
    import re

    pat = re.compile(r"traffic_bytes_per_launch\[%s\|%s\]\s*=\s*(\d+)\s*@\s*([0-9a-f]+)" % (re.escape(kernel), re.escape(workload)))
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        m = pat.search(open(path).read())
        if m:
            return int(m.group(1)) if m.group(2) == source_digest(kernel) else None
    return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return json.load(open(p)), "measured"
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


# --------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    SLOW_BITS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake"}

    def __init__(self, device_index: int, period_s: float = 0.005):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.period, self._stop, self._thr, self._h = period_s, threading.Event(), None, None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                props = torch.cuda.get_device_properties(device_index)
                bus = "%08X:%02X:%02X.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
                self._h = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.SLOW_BITS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def _events():
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def roofline(kernel, workload, bound, algo, seconds, peak, unit, peak_kind, extra=None):
    """The roofline object of one kernel: achieved = algorithmic bytes (or flops) per launch / measured
    launch time, against the measured peak; traffic from the committed ncu summary when it is current."""
    scale = 1e9 if unit == "GB/s" else 1e12
    ach = algo / seconds / scale
    r = {"kernel": kernel, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
         "peak_source": peak_kind, "algorithmic_%s_per_launch" % ("bytes" if unit == "GB/s" else "flops"): algo,
         "traffic": profile_traffic(kernel, workload)}
    if unit == "GB/s":
        r["frac_of_8000"] = ach / 8000.0
    if extra:
        r.update(extra)
    return r


def clocks_under(fn, device_index, min_ms=60.0):
    """SM clock / throttle record while `fn(i)` (one step) is repeated for at least `min_ms`: the timed
    regions themselves can be shorter than one sampling period, so the record is taken over a repeat
    of the same steps long enough to hold a dozen samples."""
    with ClockSampler(device_index) as clk:
        t0 = time.perf_counter()
        i = 0
        while (time.perf_counter() - t0) * 1e3 < min_ms:
            for _ in range(64):
                fn(i)
                i += 1
            torch.cuda.synchronize()
    return clk.summary()


def _copies_for_cold_l2(nbytes: int) -> int:
    """Number of distinct copies of a weight matrix to rotate through so that at least 8x the L2
    capacity is streamed between two uses of the same copy."""
    return max(2, -(-8 * L2_BYTES // nbytes) + 1)


# --------------------------------------------------------------------------------------------------
def build_head_workload(vt, dev, d, K, B, topk, temp, sample, seed, use_map=True, pool=16):
    """W_full -> map (from 1e7 synthetic ids through vt_build_vocab) -> W_trim copies, h pool, uniforms."""
    W_full = vt_inputs.gaussian_bf16((V, d), 0.02, seed=seed, device=dev)
    if K == V or not use_map:
        map_, W_trim = None, W_full[:K].contiguous() if K != V else W_full
    else:
        ids = vt_inputs.zipf_ids(10_000_000, V, 1.07, seed=seed + 100, noise_frac=0.05, device=dev)
        map_, _ = vt.vt_build_vocab(ids, V, K)
        W_trim = vt.vt_trim_head(W_full, map_)
        del ids
    nbytes = K * d * 2
    copies = [W_trim] + [W_trim.clone() for _ in range(_copies_for_cold_l2(nbytes) - 1)]
    if W_trim is not W_full:
        del W_full
    hs = [vt_inputs.gaussian_bf16((B, d), 1.0, seed=seed + 1000 + i, device=dev) for i in range(pool)]
    us = [vt_inputs.uniforms((B, K), seed=seed + 2000 + i, device=dev) for i in range(4)] if sample else None
    T = vt_inputs.temperatures(B, temp, temp, 0, device=dev)
    out = (torch.empty((B, 1 + topk), dtype=torch.int32, device=dev),
           torch.empty((B, 1 + topk), dtype=torch.float32, device=dev))
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD_HOST, 0, 0, K, d, B, topk), dev)
    return dict(copies=copies, map=map_, hs=hs, us=us, T=T, out=out, ws=ws, K=K, d=d, B=B, topk=topk,
                algo_bytes=K * d * 2 + B * d * 2 + (B * K * 4 if sample else 0) + 2 * B * (1 + topk) * 4)


def run_head_steps(vt, wl, steps, start=0, overlapped=True):
    """`steps` draft steps back to back on the current stream.  The weights are static during drafting,
    so the steps use vt_draft_head_overlapped: a step may start fetching W_trim while the previous
    step's last CTA is still merging.  (The very first call after the weights were written is a plain
    vt_draft_head: see time_head.)"""
    copies, hs, us = wl["copies"], wl["hs"], wl["us"]
    for i in range(start, start + steps):
        vt.vt_draft_head(hs[i % len(hs)], copies[i % len(copies)], wl["map"], wl["T"], wl["topk"],
                         us[i % len(us)] if us else None, ws=wl["ws"], out=wl["out"], overlapped=overlapped)


def first_touch(vt, wl):
    """Set-up, not warm-up: one plain step on every weight copy and every h of the pool, so that no
    buffer (nor its page-table entries) is touched for the first time inside a timed region."""
    torch.cuda.synchronize()                    # the weights were written earlier: they are final from here on
    n = max(len(wl["copies"]), len(wl["hs"]), len(wl["us"]) if wl["us"] else 0)
    run_head_steps(vt, wl, n, overlapped=False)
    torch.cuda.synchronize()


def time_head_latency(vt, wl, n=200):
    """Dependent-step latency: plain vt_draft_head calls (no overlap with the previous step), one event
    pair per call, everything enqueued ahead so that the host is not in the measured path.  Returns
    (median, p10, p90) in microseconds over n calls."""
    copies, hs, us = wl["copies"], wl["hs"], wl["us"]
    first_touch(vt, wl)
    ev = [_events() for _ in range(n)]
    for i, (e0, e1) in enumerate(ev):
        e0.record()
        vt.vt_draft_head(hs[i % len(hs)], copies[i % len(copies)], wl["map"], wl["T"], wl["topk"],
                         us[i % len(us)] if us else None, ws=wl["ws"], out=wl["out"], overlapped=False)
        e1.record()
    torch.cuda.synchronize()
    t = sorted(e0.elapsed_time(e1) * 1e3 for e0, e1 in ev[n // 10:])
    return t[len(t) // 2], t[len(t) // 10], t[(9 * len(t)) // 10]


def time_head(vt, wl, steps, warmup):
    first_touch(vt, wl)
    run_head_steps(vt, wl, warmup)
    torch.cuda.synchronize()
    e0, e1 = _events()
    e0.record()
    run_head_steps(vt, wl, steps, start=warmup)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps          # ms per step


def time_head_e2e(vt, wl, steps, warmup):
    """Same step through vt_draft_head_host: pinned host inputs, results read back every step."""
    B, K, d, topk = wl["B"], wl["K"], wl["d"], wl["topk"]
    hs = [h.cpu().pin_memory() for h in wl["hs"]]
    us = [u.cpu().pin_memory() for u in wl["us"]] if wl["us"] else None
    T = wl["T"].cpu().pin_memory()
    out = (torch.empty((B, 1 + topk), dtype=torch.int32).pin_memory(),
           torch.empty((B, 1 + topk), dtype=torch.float32).pin_memory())
    copies = wl["copies"]
    sink = 0

    def step(i):
        nonlocal sink
        vt.vt_draft_head_host(hs[i % len(hs)], copies[i % len(copies)], wl["map"], T, topk,
                              us[i % len(us)] if us else None, wl["ws"], out)
        torch.cuda.current_stream().synchronize()       # the caller consumes the ids before the next step
        sink ^= int(out[0][0, 0])

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = _events()
    e0.record()
    for i in range(warmup, warmup + steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    h2d = B * d * 2 + B * 4 + (B * K * 4 if us else 0)
    d2h = 2 * B * (1 + topk) * 4
    return e0.elapsed_time(e1) / steps, h2d, d2h


# --------------------------------------------------------------------------------------------------
def oracle_head_rate(vt, wl, seconds=12.0):
    """The CPU baseline leg: times the fp64 oracle, as it stands, on full head steps of the same workload
    for about `seconds`, and -- since its results are at hand -- compares the GPU's ids and
    log-probabilities of the same steps with them under the parity rules of the tests (ids equal unless
    the oracle's own logit margin is below 1e-3; |logp - ref| <= 2e-3).
    Returns (us per step, threads, repetitions, parity record)."""
    import numpy as np

    import oracle

    K, B, topk = wl["K"], wl["B"], wl["topk"]
    Wb = vt_inputs.bf16_bits(wl["copies"][0]).cpu().numpy().view(np.uint16)
    mh = wl["map"].cpu().numpy() if wl["map"] is not None else None
    inv = {int(v): j for j, v in enumerate(mh)} if mh is not None else None
    T = wl["T"].cpu().numpy()
    t_cpu, reps = 0.0, 0
    par = {"positions": 0, "margin_rule_accepts": 0, "mismatches": 0, "max_abs_logprob_err": 0.0}
    while True:
        i = reps % len(wl["hs"])
        hb = vt_inputs.bf16_bits(wl["hs"][i]).cpu().numpy().view(np.uint16)
        u = wl["us"][i % len(wl["us"])].cpu().numpy() if wl["us"] else None
        t0 = time.perf_counter()
        ref = oracle.draft_head(hb, Wb, mh, T, topk, u, want_full=True)
        t_cpu += time.perf_counter() - t0
        reps += 1
        gi, gl = vt.vt_draft_head(wl["hs"][i], wl["copies"][0], wl["map"], wl["T"], topk,
                                  wl["us"][i % len(wl["us"])] if wl["us"] else None, ws=wl["ws"])
        gi, gl = gi.cpu().numpy(), gl.cpu().numpy().astype(np.float64)
        for b in range(B):
            for c in range(1 + topk):
                jg = inv[int(gi[b, c])] if inv is not None else int(gi[b, c])
                jo = int(ref.trim[b, c])
                score = ref.score[b] if (c == 0 and u is not None) else ref.z[b]
                par["positions"] += 1
                if jg != jo:
                    if float(T[b]) * abs(score[jo] - score[jg]) < 1e-3:
                        par["margin_rule_accepts"] += 1
                    else:
                        par["mismatches"] += 1
                err = abs(gl[b, c] - (ref.z[b, jg] - ref.lse[b]))
                par["max_abs_logprob_err"] = max(par["max_abs_logprob_err"], float(err))
        if t_cpu >= seconds or (reps >= 3 and t_cpu >= seconds / 2):
            break
    return t_cpu / reps * 1e6, oracle.max_threads(), reps, par


def run_reference(args, rank):
    """`--impl reference`: the CPU oracle as it stands, timed on the host cores on the headline
    workload; every step is a bounded sample (a prefix of the vocabulary rows) scaled to a full step."""
    if rank != 0:
        return
    import numpy as np

    import oracle

    d, K, B, topk = HEAD["d"], HEAD["K"], HEAD["B"], HEAD["topk"]
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=1002)
    hs = [vt_inputs.gaussian_bf16((B, d), 1.0, seed=3000 + i) for i in range(8)]
    Wb = vt_inputs.bf16_bits(W).numpy().view(np.uint16)
    hb = [vt_inputs.bf16_bits(h).numpy().view(np.uint16) for h in hs]
    T = np.full(B, HEAD["temp"], dtype=np.float32)
    # calibrate rows/s, then size the per-step sample so the whole run stays near two minutes
    t0 = time.perf_counter()
    oracle.draft_head(hb[0], Wb[:4096], None, T, topk, None, want_full=False)
    per_row = (time.perf_counter() - t0) / 4096
    total_steps = args.steps + args.warmup
    rows = int(max(64, min(K, 120.0 / max(1, total_steps) / per_row)))
    Ws = np.ascontiguousarray(Wb[:rows])
    for i in range(args.warmup):
        oracle.draft_head(hb[i % 8], Ws, None, T, topk, None, want_full=False)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle.draft_head(hb[i % 8], Ws, None, T, topk, None, want_full=False)
    el = time.perf_counter() - t0
    us = el / args.steps * 1e6 * (K / rows)
    sample = "first %d of %d vocabulary rows per step, time scaled by K/rows" % (rows, K)
    line = {"impl": "reference", "metric": "drafter_lm_head_us_per_step", "value": us, "unit": "us",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": head_config(),
            "cpu_baseline": {"value": us, "unit": "us", "cores": oracle.max_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def head_config():
    return {"workload": "config2: Llama-3.2-3B-class drafter head, V=128256 d=3072 K=32768 B=1 topk=8 "
                        "T=1 greedy+top-8 (chain drafting, one vt_draft_head per step)",
            "V": V, "d": HEAD["d"], "K": HEAD["K"], "B": HEAD["B"], "topk": HEAD["topk"],
            "cold_l2": "W_trim rotated over distinct copies (>= 8x L2 streamed between reuses)",
            "launch": "vt_draft_head_overlapped (programmatic dependent launch between consecutive steps)",
            "timed_region": "CUDA events on the launching stream around exactly K steps, opened behind an untimed "
                            "0.1 ms delay kernel so that the first step's host launch latency lies outside it",
            "parallelism": "replicas"}


# --------------------------------------------------------------------------------------------------
def extras(vt, dev, peak_gbs, peak_kind):
    """K sweep of the tree-drafting head, the full-vocabulary chain head, and the vocabulary build; every
    kernel-level figure comes as a roofline object with the clocks sampled while its steps repeat."""
    out = {}
    sweep = []
    for K in TREE_KS:
        wl = build_head_workload(vt, dev, TREE["d"], K, TREE["B"], TREE["topk"], TREE["temp"], True,
                                 seed=1003)
        n = max(50, min(2000, int(0.25 / (K * TREE["d"] * 2 / 5e12))))
        ms = time_head(vt, wl, n, 20)
        lat = time_head_latency(vt, wl)
        clk = clocks_under(lambda i: run_head_steps(vt, wl, 1, start=i), dev.index)
        sweep.append({"K": K, "us_per_step": ms * 1e3, "us_dependent_step": {"median": lat[0], "p10": lat[1], "p90": lat[2]},
                      "roofline": roofline("k_head_stream", "config3 K=%d" % K, "hbm", wl["algo_bytes"], ms * 1e-3, peak_gbs,
                                           "GB/s", peak_kind),
                      "clocks": clk})
        del wl
        torch.cuda.empty_cache()
    out["tree_head_k_sweep"] = {"workload": "config3: d=4096 B=10 topk=10 T=0.7 Gumbel sampling, cold L2",
                                "points": sweep}
    out["batched_head"] = dense_case(vt, dev)
    # the paper's other drafter and task: independent 314M drafter (d=1024) and the function-calling
    # vocabulary of about 5K tokens -- heads of 10-67 MB, where the fixed cost of a launch dominates
    small = []
    for name, d_, K_ in (("independent drafter d=1024 K=32768", 1024, 32768), ("independent drafter d=1024 K=5000", 1024, 5000),
                         ("EAGLE d=3072 K=5000 (function calling)", 3072, 5000)):
        wl = build_head_workload(vt, dev, d_, K_, 1, 8, 1.0, False, seed=1007)
        ms = time_head(vt, wl, 2000, 50)
        gbs = wl["algo_bytes"] / (ms * 1e-3) / 1e9
        lat = time_head_latency(vt, wl)
        warm = dict(wl, copies=wl["copies"][:1])                      # one copy: the head stays in L2
        ms_w = time_head(vt, warm, 2000, 50)
        small.append({"workload": name + ", B=1, top-8", "mbytes": wl["algo_bytes"] / 1e6, "us_per_step_cold": ms * 1e3,
                      "gbs_cold": gbs, "frac_of_measured_cold": gbs / peak_gbs, "us_per_step_l2_resident": ms_w * 1e3,
                      "us_dependent_step_cold": {"median": lat[0], "p10": lat[1], "p90": lat[2]}})
        del wl, warm
        torch.cuda.empty_cache()
    out["small_heads"] = small
    wl = build_head_workload(vt, dev, HEAD["d"], V, HEAD["B"], HEAD["topk"], HEAD["temp"], False, seed=1002)
    ms = time_head(vt, wl, 300, 20)
    clk = clocks_under(lambda i: run_head_steps(vt, wl, 1, start=i), dev.index)
    out["full_head"] = {"workload": "config2 with the untrimmed head K=V=128256", "us_per_step": ms * 1e3,
                        "roofline": roofline("k_head_stream", "config2 K=V", "hbm", wl["algo_bytes"], ms * 1e-3, peak_gbs,
                                             "GB/s", peak_kind),
                        "clocks": clk}
    del wl
    torch.cuda.empty_cache()
    # vocabulary build at corpus scale
    n = 1_000_000_000
    ids = vt_inputs.zipf_ids(n, V, 1.07, seed=1005, noise_frac=0.05, device=dev)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_BUILD_VOCAB, n, V, 32768), dev)
    counts = torch.empty(V, dtype=torch.int32, device=dev)

    def timed(fn, reps=5, warm=2):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = _events()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    ms_h = timed(lambda: vt.vt_histogram(ids, V, counts=counts, ws=ws), reps=20, warm=3)
    clk = clocks_under(lambda i: vt.vt_histogram(ids, V, counts=counts, ws=ws), dev.index)
    vb = {"workload": "config5: 1e9 int32 ids, V=128256, 95% Zipf(1.07) + 5% uniform",
          "histogram_ms": ms_h, "histogram_gtok_s": n / (ms_h * 1e-3) / 1e9,
          "roofline": roofline("k_hist_packed", "config5 1e9 ids", "hbm", 4.0 * n, ms_h * 1e-3, peak_gbs, "GB/s", peak_kind,
                               {"note": "whole vt_histogram call (all its kernels) per 4 bytes of every id"}),
          "clocks": clk}
    vb["histogram_frac_of_measured"] = vb["roofline"]["frac"]
    for K in (8192, 32768):
        ms_b = timed(lambda: vt.vt_build_vocab(ids, V, K, ws=ws))
        vb["build_vocab_K%d_ms" % K] = ms_b
        vb["build_vocab_K%d_gtok_s" % K] = n / (ms_b * 1e-3) / 1e9
    # the selections alone, back to back on the counts of all n ids (100 calls each: the first call's start-up is
    # a tenth of a microsecond of the mean), behind a clock-sampled run of the same call: these are latency-bound
    # kernels on 8 SMs, and the histogram before them leaves the chip at the power cap's clock
    vb["select_clocks"] = clocks_under(lambda i: vt.vt_select_topk(counts, 32768, ws=ws), dev.index)
    for K in (8192, 32768):
        vb["select_topk_K%d_us" % K] = timed(lambda: vt.vt_select_topk(counts, K, ws=ws), reps=100, warm=5) * 1e3
    for p_ in (0.9, 0.99):
        vb["select_topp_p%g_us" % p_] = timed(lambda: vt.vt_select_topp(counts, p_, ws=ws), reps=100, warm=5) * 1e3
    for f_ in (1000, 100):
        vb["select_minfreq_%d_us" % f_] = timed(lambda: vt.vt_select_minfreq(counts, f_, ws=ws), reps=100, warm=5) * 1e3
    del ids
    torch.cuda.empty_cache()
    W_full = vt_inputs.gaussian_bf16((V, 4096), 0.02, seed=1006, device=dev)
    map_, _ = vt.vt_select_topk(counts, 32768, ws=ws)
    W_trim = torch.empty((32768, 4096), dtype=torch.bfloat16, device=dev)
    ms_g = timed(lambda: vt.vt_trim_head(W_full, map_, W_trim), reps=20)
    vb["trim_head_K32768_d4096_us"] = ms_g * 1e3
    vb["trim_head_roofline"] = roofline("k_gather_rows", "config5 K=32768 d=4096", "hbm", 2.0 * 32768 * 4096 * 2, ms_g * 1e-3,
                                        peak_gbs, "GB/s", peak_kind)
    out["vocab_build"] = vb
    out["draft_block"] = draft_block_case(vt, dev, timed)
    return out


def draft_block_case(vt, dev, timed):
    """The on-chip select steps around the head in a drafting block, at the paper's tree settings
    (depth 3, top-8, 32 draft tokens): three expansions + the rerank of one tree, and the greedy
    verification of 64 such trees.  Latency-bound single-CTA / warp-per-sequence kernels."""
    topk, depth, budget = 8, 3, 32
    cands = [vt_inputs.head_candidates(1 if dep == 0 else topk, topk, V, seed=1010 + dep) for dep in range(depth)]
    cands = [(i.to(dev), l.to(dev)) for i, l in cands]
    cap = topk + (depth - 1) * topk * topk
    pool = vt.tree_pool(cap, dev)

    def build_tree():
        front, base = None, 0
        for ids_, lp_ in cands:
            front = vt.vt_tree_expand(ids_, lp_, front, pool, base, topk)
            base += ids_.shape[0] * topk
        return vt.vt_tree_rerank(pool, base, budget)

    ms_t = timed(build_tree, reps=200, warm=10)
    tok, par, tgt = vt_inputs.draft_trees(64, budget, topk, V, 0.7, seed=1011)
    tok, par, tgt = tok.to(dev), par.to(dev), tgt.to(dev)
    total = torch.zeros(1, dtype=torch.int64, device=dev)
    ms_v = timed(lambda: vt.vt_verify_greedy(tok, par, tgt, tokens_total=total), reps=200, warm=10)
    out = {"workload": "tree depth 3 / top-8 / 32 draft tokens; verification of 64 trees",
           "tree_3_expansions_plus_rerank_us": ms_t * 1e3, "launches_per_tree": depth + 1,
           "verify_64_trees_us": ms_v * 1e3}
    # one tree depth of config 3 (B = 10 nodes, top-10, K = 32768): head + expansion as two launches and
    # as the single launch of vt_draft_head_expand
    wl = build_head_workload(vt, dev, TREE["d"], 32768, TREE["B"], TREE["topk"], TREE["temp"], True, seed=1003)
    B, tk = TREE["B"], TREE["topk"]
    pool2 = vt.tree_pool(64 + B * tk, dev)
    pool2[2].zero_()
    front = torch.arange(B, dtype=torch.int32, device=dev)
    copies, hs, us = wl["copies"], wl["hs"], wl["us"]
    state = {"i": 0}

    def two_launches():
        i = state["i"] = state["i"] + 1
        ids_, lp_ = vt.vt_draft_head(hs[i % len(hs)], copies[i % len(copies)], wl["map"], wl["T"], tk,
                                     us[i % len(us)], ws=wl["ws"], out=wl["out"], overlapped=True)
        vt.vt_tree_expand(ids_, lp_, front, pool2, 64, tk, col0=1)

    def one_launch():
        i = state["i"] = state["i"] + 1
        vt.vt_draft_head_expand(hs[i % len(hs)], copies[i % len(copies)], wl["map"], wl["T"], tk, us[i % len(us)],
                                front, pool2, 64, tk, ws=wl["ws"], out=wl["out"])

    out["config3_depth_K32768_head_then_expand_us"] = timed(two_launches, reps=300, warm=20) * 1e3
    out["config3_depth_K32768_fused_us"] = timed(one_launch, reps=300, warm=20) * 1e3
    return out


DENSE = dict(d=4096, K=32768, B=256, topk=8)                   # config 4: batched serving


def dense_case(vt, dev, steps=200, warmup=20):
    """Config 4: 256 rows x K=32768 x d=4096 on the tensor-core path, per-row temperatures, Gumbel sampling.
    Reported against the slower of its two bounds (tensor pipe at the measured bf16 burst rate, HBM at the
    measured copy rate)."""
    peaks, peak_kind = measured_peaks()
    d, K, B, topk = DENSE["d"], DENSE["K"], DENSE["B"], DENSE["topk"]
    wl = build_head_workload(vt, dev, d, K, B, topk, 1.0, True, seed=1004, pool=4)
    wl["T"] = vt_inputs.temperatures(B, 0.5, 1.5, seed=5001, device=dev)
    ms = time_head(vt, wl, steps, warmup)
    clk = clocks_under(lambda i: run_head_steps(vt, wl, 1, start=i), dev.index)
    st, flags, _ = wl["ws"].read_status()
    flops = 2.0 * B * K * d
    t_tensor = flops / (float(peaks["bf16_tflops"]) * 1e12) * 1e6
    t_hbm = wl["algo_bytes"] / (float(peaks["hbm_gbs"]) * 1e9) * 1e6
    if t_hbm >= t_tensor:
        roof = roofline("k_head_dense", "config4", "hbm", wl["algo_bytes"], ms * 1e-3, float(peaks["hbm_gbs"]), "GB/s", peak_kind)
    else:
        roof = roofline("k_head_dense", "config4", "tensor", flops, ms * 1e-3, float(peaks["bf16_tflops"]), "TFLOP/s", peak_kind)
    tf = flops / (ms * 1e-3) / 1e12
    return {"workload": "config4: 64 seq x 4 nodes = 256 rows, d=4096, K=32768, T_b~U[0.5,1.5], top-8, Gumbel, cold L2",
            "us_per_step": ms * 1e3, "tflops": tf, "status": st, "roofline": roof, "clocks": clk,
            "frac_of_bf16_burst": tf / float(peaks["bf16_tflops"]),
            "frac_of_bf16_sustained": tf / float(peaks["bf16_tflops_sustained"]),
            "bound_us": {"tensor_burst": t_tensor, "hbm": t_hbm},
            "frac_of_lower_bound": max(t_tensor, t_hbm) / (ms * 1e3)}


STAMP_NAMES = ("entry", "ring_requested", "released", "first_stage_landed", "last_stage_consumed", "record_written",
               "after_fence_barrier", "after_ticket", "merge_loads_done", "merge_selection_done", "merge_outputs_written")


DENSE_STAMP_NAMES = ("entry", "set_up", "released", "first_stage_landed", "mmas_issued_first_tile", "mmas_issued_last_tile",
                     "accumulators_complete_first_tile", "accumulators_complete_last_tile", "epilogue_done_first_tile",
                     "epilogue_done_last_tile", "record_written", "leaving")


def stamps_case(vt, vt_build, dev, args):
    """Where a head step's time goes: runs the headline step with the instrumented twin of the library
    (-DVT_STAMPS, built on demand) whose streaming kernel writes a nanosecond stamp per CTA and phase into
    the workspace, and prints, per launch mode, the median over launches of each phase's time after the
    first CTA was released by the launch dependency (maximum over CTAs unless said otherwise)."""
    import ctypes

    import numpy as np

    vt.LIB_PATH = vt_build.build(stamps=True)
    vt._lib = None
    L = vt.lib()
    L.vt_stamps_region.argtypes = [ctypes.c_int32] * 3 + [ctypes.c_void_p] * 3
    L.vt_stamps_region.restype = ctypes.c_int32
    shapes = {"config2": (HEAD["d"], HEAD["K"], HEAD["B"], HEAD["topk"], HEAD["temp"], False),
              "config3 K=8192": (TREE["d"], 8192, TREE["B"], TREE["topk"], TREE["temp"], True),
              "small d=1024 K=5000": (1024, 5000, 1, 8, 1.0, False)}
    for name, (d, K, B, topk, temp, sample) in shapes.items():
        wl = build_head_workload(vt, dev, d, K, B, topk, temp, sample, seed=1002)
        off, slots, ctas = ctypes.c_size_t(0), ctypes.c_int32(0), ctypes.c_int32(0)
        if not L.vt_stamps_region(B, d, topk, ctypes.byref(off), ctypes.byref(slots), ctypes.byref(ctas)):
            continue
        ws = wl["ws"]
        view = ws.buf[(ws.ptr - ws.buf.data_ptr()) + off.value:][: ctas.value * slots.value * 8].view(torch.int64)
        first_touch(vt, wl)
        rec = {"case": "stamps", "workload": name, "unit": "us after the first CTA's release, median over launches"}
        for mode, ov in (("overlapped", True), ("plain", False)):
            rows = []
            for rep_ in range(max(8, args.steps)):
                view.zero_()
                run_head_steps(vt, wl, 5, start=rep_ * 5, overlapped=ov)
                torch.cuda.synchronize()
                x = view.cpu().numpy().reshape(ctas.value, slots.value)
                x = x[x[:, 0] > 0]
                t_rel = x[:, 2].min()
                last = int(np.argmax(x[:, 8]))
                row = {"ctas": int(x.shape[0]), "entry_first": (x[:, 0].min() - t_rel) / 1e3}
                for k in range(2, 8):
                    row[STAMP_NAMES[k] + "_last"] = (x[:, k].max() - t_rel) / 1e3
                row["last_stage_consumed_median"] = float(np.median(x[:, 4] - t_rel)) / 1e3
                row["last_stage_consumed_first"] = (x[:, 4].min() - t_rel) / 1e3
                for k in range(8, 11):
                    row[STAMP_NAMES[k]] = (x[last, k] - t_rel) / 1e3
                rows.append(row)
            rec[mode] = {k: round(float(np.median([r[k] for r in rows])), 2) for k in rows[0]}
            e0, e1 = _events()
            e0.record()
            run_head_steps(vt, wl, 200, overlapped=ov)
            e1.record()
            torch.cuda.synchronize()
            rec[mode]["us_per_step_with_stamps"] = round(e0.elapsed_time(e1) * 5, 2)
        print(json.dumps(rec), flush=True)
        del wl
        torch.cuda.empty_cache()
    # the batched head (config 4): its own stamp layout, times after the first CTA's entry
    d, K, B, topk = DENSE["d"], DENSE["K"], DENSE["B"], DENSE["topk"]
    wl = build_head_workload(vt, dev, d, K, B, topk, 1.0, True, seed=1004, pool=4)
    wl["T"] = vt_inputs.temperatures(B, 0.5, 1.5, seed=5001, device=dev)
    off, slots, ctas = ctypes.c_size_t(0), ctypes.c_int32(0), ctypes.c_int32(0)
    if L.vt_stamps_region(B, d, topk, ctypes.byref(off), ctypes.byref(slots), ctypes.byref(ctas)):
        ws = wl["ws"]
        view = ws.buf[(ws.ptr - ws.buf.data_ptr()) + off.value:][: ctas.value * slots.value * 8].view(torch.int64)
        first_touch(vt, wl)
        rec = {"case": "stamps", "workload": "config4", "unit": "us after the first CTA's entry, median over launches of "
               "[median CTA, first CTA, last CTA]"}
        for mode, ov in (("overlapped", True), ("plain", False)):
            rows = []
            for rep_ in range(max(8, args.steps)):
                view.zero_()
                run_head_steps(vt, wl, 4, start=rep_ * 4, overlapped=ov)
                torch.cuda.synchronize()
                x = view.cpu().numpy().reshape(ctas.value, slots.value).astype(np.float64)
                live = x[:, 0] > 0
                t0 = x[live, 0].min()
                row = {}
                for k, nm in enumerate(DENSE_STAMP_NAMES):
                    col = x[live, k]
                    col = col[col > 0]
                    if col.size:
                        row[nm] = [(float(np.median(col)) - t0) / 1e3, (col.min() - t0) / 1e3, (col.max() - t0) / 1e3]
                row["merge_started"] = [(x[0, 12] - t0) / 1e3] * 3
                row["merge_row0_written"] = [(x[0, 13] - t0) / 1e3] * 3
                rows.append(row)
            rec[mode] = {k: [round(float(v), 2) for v in np.median(np.array([r[k] for r in rows if k in r]), axis=0)]
                         for k in rows[0]}
            e0, e1 = _events()
            e0.record()
            run_head_steps(vt, wl, 200, overlapped=ov)
            e1.record()
            torch.cuda.synchronize()
            rec[mode]["us_per_step_with_stamps"] = round(e0.elapsed_time(e1) * 5, 2)
        print(json.dumps(rec), flush=True)


def small_case(vt, dev, args, peak_gbs):
    """Short single-kernel runs sized for profiler captures (inputs larger than L2, a few launches)."""
    if args.case == "hist":
        n = args.hist_n
        ids = vt_inputs.zipf_ids(n, V, 1.07, seed=1005, noise_frac=0.05, device=dev)
        ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_BUILD_VOCAB, n, V, 32768), dev)
        counts = torch.empty(V, dtype=torch.int32, device=dev)
        for _ in range(args.warmup):
            vt.vt_histogram(ids, V, counts=counts, ws=ws)
        torch.cuda.synchronize()
        e0, e1 = _events()
        e0.record()
        for _ in range(args.steps):
            vt.vt_histogram(ids, V, counts=counts, ws=ws)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        print(json.dumps({"case": "hist", "n": n, "ms": ms, "gtok_s": n / ms / 1e6, "gbs": 4.0 * n / ms / 1e6,
                          "frac_of_measured": 4.0 * n / ms / 1e6 / peak_gbs}), flush=True)
    elif args.case == "hist-ceiling":
        # an independent, simpler kernel over the same stream (all ids folded into directly indexed 32-bit
        # bins, one shared-memory reduction per token, four loads in flight) next to the histogram proper
        n = args.hist_n
        ids = vt_inputs.zipf_ids(n, V, 1.07, seed=1005, noise_frac=0.05, device=dev)
        ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_BUILD_VOCAB, n, V, 32768), dev)
        counts = torch.empty(V, dtype=torch.int32, device=dev)
        folded = torch.empty(57344, dtype=torch.int32, device=dev)
        rec = {"case": "hist-ceiling", "n": n, "bins": 57344}
        for name, fn in (("folded", lambda: vt.vt_histogram_folded(ids, V, 57344, folded)),
                         ("histogram", lambda: vt.vt_histogram(ids, V, counts=counts, ws=ws))):
            for _ in range(args.warmup):
                fn()
            torch.cuda.synchronize()
            e0, e1 = _events()
            e0.record()
            for _ in range(args.steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            rec[name] = {"ms": ms, "gtok_s": n / ms / 1e6, "gbs": 4.0 * n / ms / 1e6, "frac_of_measured": 4.0 * n / ms / 1e6 / peak_gbs}
        rec["histogram_over_ceiling"] = rec["folded"]["ms"] / rec["histogram"]["ms"]
        print(json.dumps(rec), flush=True)
    elif args.case == "select":
        # the three selection rules on the counts of --hist-n ids of the vocabulary-build stream: Top-K first
        # (a capture of the first launches of the selection kernel sees the K = 32768 instance)
        n = args.hist_n
        ids = vt_inputs.zipf_ids(n, V, 1.07, seed=1005, noise_frac=0.05, device=dev)
        counts = vt.vt_histogram(ids, V)
        del ids
        ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, V), dev)
        rec = {"case": "select", "n": n, "V": V}
        for name, fn in (("topk_K32768_us", lambda: vt.vt_select_topk(counts, 32768, ws=ws)),
                         ("topp_p0.9_us", lambda: vt.vt_select_topp(counts, 0.9, ws=ws)),
                         ("minfreq_1000_us", lambda: vt.vt_select_minfreq(counts, 1000, ws=ws))):
            for _ in range(args.warmup):
                fn()
            torch.cuda.synchronize()
            e0, e1 = _events()
            e0.record()
            for _ in range(args.steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            rec[name] = e0.elapsed_time(e1) / args.steps * 1e3
        print(json.dumps(rec), flush=True)
    elif args.case == "dense":
        print(json.dumps(dict(case="dense", **dense_case(vt, dev, args.steps, args.warmup))), flush=True)
    else:
        wl = build_head_workload(vt, dev, TREE["d"], 32768, TREE["B"], TREE["topk"], TREE["temp"], True, seed=1003)
        ms = time_head(vt, wl, args.steps, args.warmup)
        gbs = wl["algo_bytes"] / (ms * 1e-3) / 1e9
        print(json.dumps({"case": "tree", "K": 32768, "us": ms * 1e3, "gbs": gbs,
                          "frac_of_measured": gbs / peak_gbs}), flush=True)


def max_over_ranks(ms: float, dist, dev) -> float:
    """The slowest rank's time: every rank runs an independent replica of the step (the path has no
    exchange step), so the job's time per step is the maximum over ranks.  `dist` is
    torch.distributed or None for a single process."""
    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_line(line: dict, world: int) -> dict:
    """Whole-job figures for N replicas: time per step is the slowest rank's, bandwidth adds up."""
    line["n_gpus"] = world
    line["hbm_gbs_aggregate"] = line["hbm_gbs"] * world
    return line


# --------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--case", default="head", choices=["head", "hist", "hist-ceiling", "select", "tree", "dense", "stamps"],
                    help="head: the full bench line (default); hist / select / tree / dense: a short run of the vocabulary "
                         "histogram (--hist-n ids), of the selections on its counts, of the tree-drafting head or of the batched head, for profiler "
                         "captures; stamps: per-phase timeline of a head step from the instrumented build")
    ap.add_argument("--hist-n", type=int, default=200_000_000)
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    import paper_2506_22694_b200 as vt
    from paper_2506_22694_b200 import build as vt_build

    vt_build.build()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    peaks, peak_kind = measured_peaks()
    peak_gbs = float(peaks["hbm_gbs"])
    if args.case == "stamps":
        stamps_case(vt, vt_build, dev, args)
        return
    if args.case != "head":
        small_case(vt, dev, args, peak_gbs)
        return
    wl = build_head_workload(vt, dev, HEAD["d"], HEAD["K"], HEAD["B"], HEAD["topk"], HEAD["temp"], False,
                             seed=1002)
    first_touch(vt, wl)                          # set-up: every weight copy and every h has been used once

    def bracketed(n, start):
        """n steps between two events on the launching stream.  The region opens on the device behind an
        untimed delay kernel (about 0.1 ms of torch's spin kernel): the host has queued the first steps by
        then, so what the events bracket is n steps of device time and not the host's latency in launching
        the first of them into an idle GPU."""
        e0, e1 = _events()
        torch.cuda._sleep(200_000)
        e0.record()
        run_head_steps(vt, wl, n, start=start)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    bracketed(args.warmup, 0)                    # the W warm-up steps take the same path as the timed ones
    if dist:
        dist.barrier()
    launches0 = vt.launch_count()
    torch.cuda.synchronize()
    elapsed_ms = bracketed(args.steps, args.warmup)
    launches = vt.launch_count() - launches0
    if dist:
        dist.barrier()
    ms_step = max_over_ranks(elapsed_ms, dist, dev) / args.steps
    # clocks: sampled while the same steps repeat for a few dozen milliseconds (the timed region above can
    # be shorter than one sampling period)
    clocks = clocks_under(lambda i: run_head_steps(vt, wl, 1, start=i), local)
    lat = time_head_latency(vt, wl)
    lat_ms = max_over_ranks(lat[0], dist, dev)
    e2e_ms, h2d, d2h = time_head_e2e(vt, wl, max(200, min(args.steps, 5000)), 50)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    st, flags, _ = wl["ws"].read_status()
    if st != 0:
        raise SystemExit("device-side status after the timed region: %s (flags %d)" % (vt.status_str(st), flags))

    roof = roofline("k_head_stream", "config2", "hbm", wl["algo_bytes"], ms_step * 1e-3, peak_gbs, "GB/s", peak_kind)
    line = {
        "metric": "drafter_lm_head_us_per_step", "value": ms_step * 1e3, "unit": "us", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": head_config(),
        "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches), "clocks": clocks,
        "hbm_gbs": roof["achieved"],
        "roofline": roof,
        "dependent_step": {"what": "plain vt_draft_head, one event pair per call, nothing overlapped with the previous step",
                           "us_median": lat_ms, "us_p10": lat[1], "us_p90": lat[2],
                           "frac_of_measured_hbm": wl["algo_bytes"] / (lat_ms * 1e-6) / 1e9 / peak_gbs},
    }
    line = aggregate_line(line, world)
    if rank == 0 and world == 1:
        if not args.no_cpu_baseline:
            us, threads, reps, par = oracle_head_rate(vt, wl, seconds=12.0)
            line["cpu_baseline"] = {"value": us, "unit": "us", "cores": threads, "kind": "oracle",
                                    "sample": "%d full head steps (all %d rows) of the same workload" % (reps, wl["K"])}
            line["parity_slack"] = par
        del wl
        torch.cuda.empty_cache()
        if not args.no_extras:
            line.update(extras(vt, dev, peak_gbs, peak_kind))
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the clustered-head-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 2|3|4]

One *step* is one decode step of the whole model-shaped workload: the L per-layer
chai_decode_attention calls for one new token per request, enqueued back to back on one stream.
All layers' caches are resident in HBM, each layer has its own buffers, and one layer's working set
(>= 168 MiB) already exceeds L2, so every step streams from DRAM.  The headline value is algorithmic
bytes per step / step time (GB/s); microseconds per step ride along.  The same run also times
clustered prefill (workload 5) and K-cache compaction (workload 4's shape) and reports them as
extra objects of the one JSON line.

With N > 1 (torchrun) every rank runs an independent replica of the workload on its own GPU: the
path has no exchange step, so there is no collective on the data path; the barrier and the
max-over-ranks reduction are the only communication.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2403_08058_b200 import chai, replicas, synth  # noqa: E402

METRIC = "clustered decode attention: algorithmic HBM GB/s over one decode step (us/step alongside)"
UNIT = "GB/s"


TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "decode_persistent_kernel_dram_traffic.json")


def load_traffic_ratio():
    """DRAM bytes per launch over algorithmic bytes per launch of the decode kernel, as measured by the ncu capture
    recorded in profiles/ (written by `bench.py --record-traffic`, which parses that capture); None when absent."""
    try:
        rec = json.load(open(TRAFFIC_RECORD))
        return float(rec["dram_bytes_per_launch"]) / float(rec["algorithmic_bytes_per_launch"]), rec
    except (OSError, ValueError, KeyError, ZeroDivisionError):
        return None, None


def record_traffic(csv_path: str, layers: int, workload: int):
    """Turns an ncu CSV (--page raw, or --csv log of --metrics dram__bytes_read.sum,dram__bytes_write.sum) of
    `bench.py --workload W --layers N --skip-extras` into the tracked record: mean DRAM bytes per captured launch of
    the decode kernel beside the mean algorithmic bytes of the same layers."""
    import csv
    rows = list(csv.reader(open(csv_path, errors="replace")))
    hdr_i = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    hdr = rows[hdr_i]
    per_launch = {}
    if "Metric Name" in hdr:          # one row per (launch, metric)
        ki, mi, vi, ui, idi = (hdr.index(n) for n in ("Kernel Name", "Metric Name", "Metric Value", "Metric Unit", "ID"))
        for r in rows[hdr_i + 1:]:
            if len(r) <= vi or "decode_persistent_kernel" not in r[ki] or not r[mi].startswith("dram__bytes_"):
                continue
            unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[r[ui]]
            per_launch[r[idi]] = per_launch.get(r[idi], 0.0) + float(r[vi].replace(",", "")) * unit
    else:                             # raw page: one row per launch, one column per metric, units in the next row
        units = rows[hdr_i + 1]
        ki = hdr.index("Kernel Name")
        cols = [i for i, n in enumerate(hdr) if n in ("dram__bytes_read.sum", "dram__bytes_write.sum")]
        for j, r in enumerate(rows[hdr_i + 2:]):
            if len(r) <= max(cols) or "decode_persistent_kernel" not in r[ki]:
                continue
            per_launch[j] = sum(float(r[i].replace(",", "")) * {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[units[i]]
                                for i in cols)
    if not per_launch:
        raise SystemExit("no decode_persistent_kernel launches with dram__bytes_* metrics in " + csv_path)
    w = synth.WORKLOADS[workload]
    es = 2 if w.dtype == "bf16" else 4
    ks = [min(synth.layer_k(workload, layer, 0), w.H) for layer in range(min(layers, w.layers))]
    alg = float(np.mean([decode_bytes(w.B, w.H, k, w.T, w.D, es) for k in ks]))
    rec = {"kernel": "decode_persistent_kernel", "workload": f"{w.name}, first {len(ks)} layers (k = {ks})",
           "launches_captured": len(per_launch), "dram_bytes_per_launch": float(np.mean(list(per_launch.values()))),
           "algorithmic_bytes_per_launch": alg,
           "how": f"`python bench.py --workload {workload} --layers {layers} --skip-extras --no-graph --steps 3 --warmup 3` "
                  "(exit 0), then the same command under `ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum "
                  "--clock-control none -k regex:decode_persistent -s 8 -c 12 --csv --log-file traffic.csv`, then "
                  f"`python bench.py --record-traffic traffic.csv --workload {workload} --layers {layers}`"}
    rec["ratio"] = rec["dram_bytes_per_launch"] / alg
    json.dump(rec, open(TRAFFIC_RECORD, "w"), indent=1)
    print(json.dumps(rec))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), tf_burst=float(p["bf16_tflops"]),
                    tf_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz, self.power = [], set(), None, []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:  # NVML missing: clocks are reported as unknown
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                except Exception:
                    pass
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return dict(sm_mhz=(statistics.median(self.samples) if self.samples else None), sm_max_mhz=self.max_mhz,
                    reasons=sorted(self.reasons), samples=len(self.samples),
                    power_w=(statistics.median(self.power) if self.power else None))


def decode_bytes(B, H, k, T, D, es):
    """Algorithmic bytes of one layer's decode call: (k+H) cache planes, the representatives' query rows,
    the outputs and the two maps."""
    return (k + H) * B * T * D * es + k * B * D * es + H * B * D * es + 4 * B * (H + k)


def prefill_flops(B, H, k, T, D):
    """Causal pairs only: one QK^T per cluster and one PV per head, 2*D flops per (row, key) pair each."""
    return 2 * D * (T * (T + 1) // 2) * (k + H) * B


class DecodeWorkload:
    def __init__(self, cfg_id: int, device, seed: int = 0, layers: int | None = None):
        w = synth.WORKLOADS[cfg_id]
        if layers:
            import dataclasses
            w = dataclasses.replace(w, layers=min(layers, w.layers))
        self.w, self.cfg_id, self.device = w, cfg_id, device
        self.layers = []
        self.es = 2 if w.dtype == "bf16" else 4
        self.dt = chai.CHAI_BF16 if w.dtype == "bf16" else chai.CHAI_F32
        ws_bytes = 0
        for layer in range(w.layers):
            c = synth.decode_layer(cfg_id, layer, seed, device=device, with_k_full=False)
            c["out"] = torch.empty_like(c["q"])
            ws_bytes = max(ws_bytes, chai.chai_decode_workspace_bytes(w.B, w.H, c["k"], w.T, w.D, self.dt))
            self.layers.append(c)
        self.ws = chai.new_workspace(ws_bytes, device)
        self.bytes_per_layer = [decode_bytes(w.B, w.H, c["k"], w.T, w.D, self.es) for c in self.layers]
        self.bytes_per_step = sum(self.bytes_per_layer)
        self.launches_per_step = w.layers  # one persistent kernel per layer call

    def step(self):
        for c in self.layers:
            chai.chai_decode_attention(c["q"], c["k_rep"], c["v"], c["membership"], c["reps"], c["scale"], out=c["out"],
                                       workspace=self.ws)

    def step_with_events(self, events):
        events[0].record()
        for i, c in enumerate(self.layers):
            chai.chai_decode_attention(c["q"], c["k_rep"], c["v"], c["membership"], c["reps"], c["scale"], out=c["out"],
                                       workspace=self.ws)
            events[i + 1].record()

    def make_host_buffers(self):
        self.q_host = [c["q"].cpu().pin_memory() for c in self.layers]
        self.o_host = [torch.empty_like(q).pin_memory() for q in self.q_host]
        self.q_stage = torch.empty_like(self.layers[0]["q"])
        self.o_stage = torch.empty_like(self.layers[0]["q"])

    def step_host(self):
        """One decode step through the host-buffer entry: every layer call enqueues upload, kernel and download;
        the host waits once, at the end of the step, for the outputs to have landed."""
        for c, qh, oh in zip(self.layers, self.q_host, self.o_host):
            chai.chai_decode_attention_host_async(qh, oh, self.q_stage, self.o_stage, c["k_rep"], c["v"],
                                                  c["membership"], c["reps"], c["scale"], self.ws)
        torch.cuda.current_stream().synchronize()

    def make_pipeline(self):
        self.s_up, self.s_comp, self.s_down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        self.q_stages = [torch.empty_like(c["q"]) for c in self.layers]
        self.o_stages = [torch.empty_like(c["q"]) for c in self.layers]
        self.ev_up = [torch.cuda.Event() for _ in self.layers]
        self.ev_k = [torch.cuda.Event() for _ in self.layers]

    def step_host_pipelined(self):
        """The step through chai_decode_attention_host_streams: every layer call spreads its upload, kernels and
        download over three streams, a staging buffer per layer; the host waits once at the end of the step."""
        for i, (c, qh, oh) in enumerate(zip(self.layers, self.q_host, self.o_host)):
            chai.chai_decode_attention_host_streams(qh, oh, self.q_stages[i], self.o_stages[i], c["k_rep"], c["v"],
                                                    c["membership"], c["reps"], c["scale"], self.ws, self.s_comp,
                                                    self.s_up, self.s_down, self.ev_up[i], self.ev_k[i])
        self.s_down.synchronize()   # the downloads come last; the other two streams have drained by then
        self.s_comp.synchronize()
        self.s_up.synchronize()

    def step_host_blocking(self):
        """The same with the blocking entry: the host waits after every layer call."""
        for c, qh, oh in zip(self.layers, self.q_host, self.o_host):
            chai.chai_decode_attention_host(qh, oh, self.q_stage, self.o_stage, c["k_rep"], c["v"], c["membership"],
                                            c["reps"], c["scale"], self.ws)


def time_region(fn, steps, sync_all):
    """Times `steps` calls of fn with CUDA events on the current stream; barrier + synchronize on both sides."""
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    sync_all()
    return ms


def cpu_baseline_decode(cfg_id: int, seed: int, budget_s: float = 12.0):
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload: whole layers of
    the decode step, request by request, until about `budget_s` seconds of oracle time are spent."""
    from oracle import chai_oracle as orc
    w = synth.WORKLOADS[cfg_id]
    es = 2 if w.dtype == "bf16" else 4
    spent, nbytes, n_req, layer, wall0 = 0.0, 0, 0, 0, time.perf_counter()
    # oracle time is the timed quantity; generation and widening are not, so the wall clock is bounded too
    while spent < budget_s and layer < w.layers and time.perf_counter() - wall0 < 60.0:
        c = synth.decode_layer(cfg_id, layer, seed, device="cpu", B=2, with_k_full=False)
        args = [orc._f64(c[n]) for n in ("q", "k_rep", "v")]
        reps_run = 0
        while reps_run < 40 and spent < budget_s:
            t0 = time.perf_counter()
            orc.cha_attention(args[0], args[1], args[2], c["membership"], c["reps"], c["scale"], causal=False)
            spent += time.perf_counter() - t0
            nbytes += decode_bytes(2, w.H, c["k"], w.T, w.D, es)
            n_req += 2
            reps_run += 1
        layer += 1
    return dict(value=nbytes / spent / 1e9, unit=UNIT, cores=orc.num_threads(), kind="oracle",
                sample=f"first {layer} layers x 2 requests of workload {cfg_id}, each up to 40 times ({n_req} request-layers, "
                       f"{spent:.1f} s of oracle time, inputs already widened to fp64)", seconds=spent)


def cpu_baseline_prefill(seed: int = 0, budget_s: float = 12.0):
    """Times the CPU oracle, as it stands, on workload 5 itself: whole requests (all rows, all heads), one after
    the other and round again until about `budget_s` seconds of oracle time are spent.  Flops counted as for the
    GPU: 2*D per causal (row, key) pair, once per cluster for the scores and once per head for the values."""
    from oracle import chai_oracle as orc
    case = synth.prefill_case(seed=seed, device="cpu")
    B, H, T, D, k = case["B"], case["H"], case["T"], case["D"], case["k"]
    mem, reps = case["membership"], case["reps"]
    idx = reps.long()[:, :, None, None].expand(B, k, T, D)
    k_rep = torch.gather(case["k_full"], 1, idx)
    wide = [[orc._f64(x[b:b + 1]) for x in (case["q_full"], k_rep, case["v"])] for b in range(B)]
    spent, flops, n_req = 0.0, 0.0, 0
    wall0 = time.perf_counter()
    while spent < budget_s and time.perf_counter() - wall0 < 90.0:
        b = n_req % B
        t0 = time.perf_counter()
        orc.cha_attention(wide[b][0], wide[b][1], wide[b][2], mem[b:b + 1], reps[b:b + 1], case["scale"], True)
        spent += time.perf_counter() - t0
        flops += prefill_flops(1, H, k, T, D)
        n_req += 1
    return dict(value=flops / spent / 1e12, unit="TFLOP/s", cores=orc.num_threads(), kind="oracle",
                sample=f"{n_req} whole requests of workload 5 (its {B} requests in rotation; {spent:.1f} s of oracle time, "
                       "fp64, inputs already widened)", seconds=spent)


def run_reference(args, rank):
    """The reference arm of this tier is the CPU oracle timed on the host cores."""
    if rank != 0:
        return
    from oracle import chai_oracle as orc
    cfg_id = args.workload
    w = synth.WORKLOADS[cfg_id]
    es = 2 if w.dtype == "bf16" else 4
    c = synth.decode_layer(cfg_id, 0, 0, device="cpu", B=2, with_k_full=False)
    a = [orc._f64(c[n]) for n in ("q", "k_rep", "v")]
    nbytes = decode_bytes(2, w.H, c["k"], w.T, w.D, es)

    def step():
        orc.cha_attention(a[0], a[1], a[2], c["membership"], c["reps"], c["scale"], causal=False)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = nbytes * args.steps / dt / 1e9
    sample = f"each step = layer 0, 2 of {w.B} requests of workload {cfg_id} (fp64 oracle, inputs pre-widened)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def bench_prefill(device, peaks, iters=20, warmup=3):
    case = synth.prefill_case(seed=0, device=device)
    B, H, T, D, k = case["B"], case["H"], case["T"], case["D"], case["k"]
    k_rep = chai.chai_compact_k_cache(case["k_full"], case["reps"])
    ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(B, H, k, T, D, chai.CHAI_BF16), device)
    out = torch.empty_like(case["q_full"])
    feats = torch.empty((B, H, 25), device=device, dtype=torch.float32)

    def attn():
        chai.chai_prefill_attention(case["q_full"], k_rep, case["v"], case["membership"], case["reps"], case["scale"],
                                    True, out=out, workspace=ws)

    def flow():
        chai.chai_prefix_features(case["q_full"], case["k_full"], 5, case["scale"], features=feats)
        mem, reps, _, _ = chai.chai_cluster_heads(feats, k, 20, 0, want_inertia=False)
        chai.chai_compact_k_cache(case["k_full"], reps, k_rep=k_rep)
        chai.chai_prefill_attention(case["q_full"], k_rep, case["v"], mem, reps, case["scale"], True, out=out,
                                    workspace=ws)

    res = {}
    for name, fn in (("attention", attn), ("flow", flow)):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        # calls enqueued back to back, one pair of events around all of them (launch latency overlaps the
        # previous call, as in a serving loop); every call streams its 168 MB working set again
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        res[name] = e0.elapsed_time(e1) / iters
    fl = prefill_flops(B, H, k, T, D)
    tf = fl / (res["attention"] * 1e-3) / 1e12
    # the same kernel on longer prompts (same heads and clusters): items are longer, so the per-item and
    # per-launch costs weigh less; reported beside the headline workload, not instead of it
    longer = {}
    for Bl, Tl in ((2, 4096), (1, 8192), (1, 16384)):
        cl = synth.prefill_case(seed=0, B=Bl, T=Tl, device=device)
        krl = chai.chai_compact_k_cache(cl["k_full"], cl["reps"])
        del cl["k_full"]
        wsl = chai.new_workspace(chai.chai_prefill_workspace_bytes(Bl, H, k, Tl, D, chai.CHAI_BF16), device)
        outl = torch.empty_like(cl["q_full"])
        call = lambda: chai.chai_prefill_attention(cl["q_full"], krl, cl["v"], cl["membership"], cl["reps"], cl["scale"],
                                                   True, out=outl, workspace=wsl)
        for _ in range(warmup):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(10):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms_l = e0.elapsed_time(e1) / 10
        tf_l = prefill_flops(Bl, H, k, Tl, D) / (ms_l * 1e-3) / 1e12
        longer[f"B{Bl}_T{Tl}"] = {"ms": ms_l, "tflops": tf_l, "frac_of_burst_peak": tf_l / peaks["tf_burst"]}
        del cl, krl, outl, wsl
        torch.cuda.empty_cache()
    # the same call repeated for about a second, clocks and power sampled meanwhile: this kernel runs at the
    # board's power cap, so the sustained figure (against the sustained cuBLAS peak) belongs beside the burst one
    n_sust = max(200, int(1.0 / (res["attention"] * 1e-3)))
    with ClockSampler(torch.cuda.current_device()) as clk:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_sust):
            attn()
        e1.record()
        torch.cuda.synchronize()
    ms_sust = e0.elapsed_time(e1) / n_sust
    tf_sust = fl / (ms_sust * 1e-3) / 1e12
    return {
        "longer_prompts": longer,
        "workload": synth.WORKLOADS[5].name, "ms_attention": res["attention"], "ms_flow_features_kmeans_compact_attention": res["flow"],
        "algorithmic_gflop": fl / 1e9, "tflops": tf,
        "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["tf_burst"], "unit": "TFLOP/s",
                     "frac": tf / peaks["tf_burst"], "peak_source": peaks["source"] + " (burst: kernel timed alone)",
                     "traffic": None},
        "sustained": {"calls": n_sust, "ms_attention": ms_sust, "tflops": tf_sust, "peak": peaks["tf_sustained"],
                      "frac": tf_sust / peaks["tf_sustained"], "peak_source": peaks["source"] + " (sustained)",
                      "clocks": clk.summary()},
        "l2": "working set 168 MB per call exceeds L2",
    }


def bench_compaction(device, peaks, iters=20, warmup=3):
    """Out-of-place compaction of one workload-4 layer for k = 12, 24 and 36 (the range that workload draws from),
    layer after layer over six layers' caches (1.2 GB, far more than L2), as a model's 64 layers are compacted one
    after the other; and, for k = 24, the same call after a 256 MB write that leaves L2 full of dirty lines, which
    the call then has to evict."""
    w = synth.WORKLOADS[4]
    sets = 6
    g = torch.Generator(device=device).manual_seed(4)
    k_full = [torch.randn((w.B, w.H, w.T, w.D), device=device, generator=g).to(torch.bfloat16) for _ in range(sets)]

    def timed(k, reps, k_rep, flush):
        ts = []
        for i in range(warmup + iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if flush is not None:  # one call, right behind the write that fills L2
                flush.fill_(i & 1)
                e0.record()
                chai.chai_compact_k_cache(k_full[i % sets], reps, k_rep=k_rep[i % sets])
                e1.record()
                n = 1
            else:                  # the six layers back to back, as a model's layers are compacted
                e0.record()
                for j in range(sets):
                    chai.chai_compact_k_cache(k_full[j], reps, k_rep=k_rep[j])
                e1.record()
                n = sets
            torch.cuda.synchronize()
            if i >= warmup:
                ts.append(e0.elapsed_time(e1) / n)
        return statistics.median(ts)

    by_k = {}
    for k in (12, 24, 36):
        _, reps = synth.batch_partitions(w.B, w.H, k, "uneven", 0, 4, 0)
        reps = torch.as_tensor(reps, device=device)
        k_rep = [torch.empty((w.B, k, w.T, w.D), device=device, dtype=torch.bfloat16) for _ in range(sets)]
        nbytes = 2 * k * w.B * w.T * w.D * 2
        ms = timed(k, reps, k_rep, None)
        gbs = nbytes / (ms * 1e-3) / 1e9
        by_k[f"k{k}"] = {"us": ms * 1e3, "algorithmic_mb": nbytes / 1e6, "gbs": gbs, "frac": gbs / peaks["hbm"]}
        if k == 24:
            ms_dirty = timed(k, reps, k_rep, torch.empty(256 << 20, device=device, dtype=torch.uint8))
            dirty = {"us": ms_dirty * 1e3, "gbs": nbytes / (ms_dirty * 1e-3) / 1e9,
                     "note": "L2 full of the flush's dirty lines, which the call evicts"}
        del k_rep
    mid = by_k["k24"]
    return {"workload": "config4 one layer (B 4, H 72, T 2048, D 128), k = 12 / 24 / 36", "by_k": by_k,
            "us": mid["us"], "algorithmic_mb": mid["algorithmic_mb"], "gbs": mid["gbs"],
            "roofline": {"bound": "hbm", "achieved": mid["gbs"], "peak": peaks["hbm"], "unit": "GB/s", "frac": mid["frac"],
                         "peak_source": peaks["source"], "traffic": None, "workload": "k = 24"},
            "l2": "six layers' caches in rotation (1.2 GB): every call reads and writes memory that is not in L2",
            "after_a_256MB_write": dirty}


def bench_serving(device, peaks, iters=20, warmup=3):
    """The serving-shaped steps at workload 2's layer shape (k = 8): a ragged batch whose lengths are spread
    over 1/4..1 of the capacity, read from a cache that was compacted in place; the per-token append; the
    in-place compaction itself."""
    w = synth.WORKLOADS[2]
    k, B, H, T_cap, D, es = 8, w.B, w.H, w.T, w.D, 2
    c = synth.decode_layer(2, 0, 1, device=device, B=B, H=H, T=T_cap, k=k, with_k_full=True)
    rng = np.random.default_rng(7)
    lens = rng.integers(T_cap // 4, T_cap, size=B).astype(np.int32)
    lens[0] = T_cap - 1
    seq = torch.as_tensor(lens, device=device)
    reps_host = c["reps"].cpu().numpy()
    cache = c["k_full"].clone()
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(B, H, k, T_cap, D, chai.CHAI_BF16), device)
    flush = torch.empty(256 << 20, device=device, dtype=torch.uint8)

    def timed(fn, before=None):
        ts = []
        for i in range(warmup + iters):
            if before is not None:
                before()
            flush.fill_(i & 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if i >= warmup:
                ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)

    # in-place compaction (restore the full cache before every run)
    ms_c = timed(lambda: chai.chai_compact_k_cache_inplace(cache, c["reps"], T=T_cap), before=lambda: cache.copy_(c["k_full"]))
    moved = int(sum(1 for b in range(B) for cc in range(k) if reps_host[b, cc] >= 0 and reps_host[b, cc] != cc))
    bytes_c = 2 * moved * T_cap * D * es
    # ragged decode from the strided cache
    out = torch.empty_like(c["q"])
    ms_d = timed(lambda: chai.chai_decode_attention_ragged(c["q"], cache, c["v"], c["membership"], c["reps"], seq, c["scale"],
                                                           T_max=T_cap, out=out, workspace=ws))
    bytes_d = int(sum((k + H) * int(n) * D * es for n in lens)) + (k + H) * B * D * es
    # the same call with every request at full length, timed the same way (single call after an L2 flush,
    # launch latency included), as the yardstick for the ragged number
    full = torch.full((B,), T_cap, dtype=torch.int32, device=device)
    ms_f = timed(lambda: chai.chai_decode_attention_ragged(c["q"], cache, c["v"], c["membership"], c["reps"], full, c["scale"],
                                                           T_max=T_cap, out=out, workspace=ws))
    bytes_f = (k + H) * B * T_cap * D * es + (k + H) * B * D * es
    # the same two calls timed like the headline: back to back over four cache sets (2 GB: every call streams its
    # own caches from DRAM), launch latency hidden behind the previous call
    sets = [(cache, c["v"])] + [(torch.randn_like(cache), torch.randn_like(c["v"])) for _ in range(3)]

    def back_to_back(lens_t):
        def run():
            for kc_, vc_ in sets:
                chai.chai_decode_attention_ragged(c["q"], kc_, vc_, c["membership"], c["reps"], lens_t, c["scale"],
                                                  T_max=T_cap, out=out, workspace=ws)
        for _ in range(warmup):
            run()
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()          # as in the headline: the calls captured once and replayed
        with torch.cuda.graph(graph, stream=side):
            for _ in range(5):
                run()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters // 5):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / ((iters // 5) * 5 * len(sets))

    ms_d_b2b, ms_f_b2b = back_to_back(seq), back_to_back(full)
    # equal lengths that end exactly on a 128-row tile, one row short of it and one row past it: a ragged last tile
    # must cost what its bytes cost (it once cost several full tiles)
    tail_check = {}
    for n in (T_cap - 641, T_cap - 640, T_cap - 639):
        tail_check[str(n)] = back_to_back(torch.full((B,), n, dtype=torch.int32, device=device)) * 1e3
    del sets
    # append (no advance, so every run writes the same rows)
    k_new = torch.randn((B, H, D), device=device).to(torch.bfloat16)
    v_new = torch.randn((B, H, D), device=device).to(torch.bfloat16)
    ms_a = timed(lambda: chai.chai_append_kv(k_new, v_new, cache, c["v"], c["reps"], seq, advance=False))
    gbs_d, gbs_c = bytes_d / (ms_d * 1e-3) / 1e9, bytes_c / (ms_c * 1e-3) / 1e9
    # one request with a 128k-token context (k = 8): 1.3 GB per layer call, timed the same way
    del c, cache
    torch.cuda.empty_cache()
    TL = 131072
    cl = synth.decode_layer(2, 1, 3, device=device, B=1, H=H, T=TL, k=k, with_k_full=False)
    wsl = chai.new_workspace(chai.chai_decode_workspace_bytes(1, H, k, TL, D, chai.CHAI_BF16), device)
    outl = torch.empty_like(cl["q"])
    ms_l = timed(lambda: chai.chai_decode_attention(cl["q"], cl["k_rep"], cl["v"], cl["membership"], cl["reps"], cl["scale"],
                                                    out=outl, workspace=wsl))
    bytes_l = decode_bytes(1, H, k, TL, D, es)
    gbs_l = bytes_l / (ms_l * 1e-3) / 1e9
    long_ctx = {"workload": "B 1, H 32, k 8, T 131072, bf16", "us": ms_l * 1e3, "algorithmic_mb": bytes_l / 1e6, "gbs": gbs_l,
                "roofline": {"bound": "hbm", "achieved": gbs_l, "peak": peaks["hbm"], "unit": "GB/s",
                             "frac": gbs_l / peaks["hbm"], "peak_source": peaks["source"], "traffic": None}}
    del cl
    return {"workload": "config2 layer shape, k=8, lengths uniform in [T/4, T), K cache compacted in place",
            "long_context_decode": long_ctx,
            "seq_lens": [int(x) for x in lens],
            "full_length_same_timing": {"us": ms_f * 1e3, "algorithmic_mb": bytes_f / 1e6, "gbs": bytes_f / (ms_f * 1e-3) / 1e9},
            "ragged_decode": {"us": ms_d * 1e3, "algorithmic_mb": bytes_d / 1e6, "gbs": gbs_d,
                              "roofline": {"bound": "hbm", "achieved": gbs_d, "peak": peaks["hbm"], "unit": "GB/s",
                                           "frac": gbs_d / peaks["hbm"], "peak_source": peaks["source"], "traffic": None},
                              "back_to_back": {"us": ms_d_b2b * 1e3, "gbs": bytes_d / (ms_d_b2b * 1e-3) / 1e9,
                                               "frac": bytes_d / (ms_d_b2b * 1e-3) / 1e9 / peaks["hbm"],
                                               "full_length_us": ms_f_b2b * 1e3,
                                               "full_length_gbs": bytes_f / (ms_f_b2b * 1e-3) / 1e9,
                                               "us_over_full_length_us_times_byte_ratio": ms_d_b2b / (ms_f_b2b * bytes_d / bytes_f),
                                               "equal_lengths_us": tail_check,
                                               "note": "four cache sets in rotation, the calls captured in a CUDA graph and replayed"}},
            "compact_inplace": {"us": ms_c * 1e3, "planes_moved": moved, "algorithmic_mb": bytes_c / 1e6, "gbs": gbs_c,
                                "roofline": {"bound": "hbm", "achieved": gbs_c, "peak": peaks["hbm"], "unit": "GB/s",
                                             "frac": gbs_c / peaks["hbm"], "peak_source": peaks["source"], "traffic": None}},
            "append_kv": {"us": ms_a * 1e3, "bytes": 2 * (H + k) * B * D * es, "bound": "latency (one CTA per request)"},
            "l2": "flushed by a 256 MB write before every timed call"}


def bench_config1(device, iters=200, warmup=10):
    """Configuration 1 (fp32, B 1, H 32, k 8, T 256, D 128; 5 MB, L2 resident): a latency point, microseconds only.
    The decode call and the clustering of its [1,32,64] features, back to back on one stream; beside them the
    oracle on one host thread."""
    c = synth.decode_layer(1, 0, 0, device=device, with_k_full=False)
    ws = chai.new_workspace(chai.chai_decode_workspace_bytes(c["B"], c["H"], c["k"], c["T"], c["D"], chai.CHAI_F32), device)
    out = torch.empty_like(c["q"])
    feats_np, _, _ = synth.blob_features(B=1, H=32, F=64, k=8, seed=0)
    feats = torch.as_tensor(feats_np, device=device)
    dec = lambda: chai.chai_decode_attention(c["q"], c["k_rep"], c["v"], c["membership"], c["reps"], c["scale"], out=out,
                                             workspace=ws)
    km = lambda: chai.chai_cluster_heads(feats, 8, 20, 0, want_inertia=False)
    res = {"workload": "config1: fp32, B 1, H 32, k 8, T 256, D 128 (L2 resident); features [1,32,64]"}
    for name, fn in (("decode", dec), ("cluster_heads", km)):
        for _ in range(warmup):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        res[name + "_us_eager"] = e0.elapsed_time(e1) * 1e3 / iters
        # the same 20 calls captured in a CUDA graph: what the GPU needs without the host's share
        g = torch.cuda.CUDAGraph()
        st = torch.cuda.Stream()
        st.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=st):
            for _ in range(20):
                fn()
        g.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(10):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        res[name + "_us_graph"] = e0.elapsed_time(e1) * 1e3 / 200
    res["note"] = ("eager: calls enqueued back to back from Python (launch and binding latency); graph: 20 calls per "
                   "captured graph, replayed")
    from oracle import chai_oracle as orc
    cpu = {n: c[n].cpu() for n in ("q", "k_rep", "v", "membership", "reps")}
    # one host thread for the oracle: the OpenMP runtime is told so from here (the oracle itself is left as it is)
    threads_before, gomp = orc.num_threads(), None
    try:
        import ctypes
        gomp = ctypes.CDLL("libgomp.so.1")
        gomp.omp_set_num_threads(1)
    except OSError:
        gomp = None
    orc.cha_attention(cpu["q"], cpu["k_rep"], cpu["v"], cpu["membership"], cpu["reps"], c["scale"], False)
    t0 = time.perf_counter()
    n = 0
    while time.perf_counter() - t0 < 0.5:
        orc.cha_attention(cpu["q"], cpu["k_rep"], cpu["v"], cpu["membership"], cpu["reps"], c["scale"], False)
        n += 1
    res["oracle_decode_us"] = (time.perf_counter() - t0) * 1e6 / n
    res["oracle_threads"] = orc.num_threads()
    if gomp is not None:
        gomp.omp_set_num_threads(threads_before)
    return res


def bench_fp8(device, peaks, iters=20, warmup=3):
    """Decode on e4m3 caches at workload 2's layer shape for k = 8 and k = 32: the layer calls run back to back over
    eight different cache sets (1.3 - 2.2 GB, larger than L2), as in the main decode number."""
    w = synth.WORKLOADS[2]
    B, H, T, D = w.B, w.H, w.T, w.D
    res = {}
    for k in (8, 32):
        sets = []
        for i in range(8):
            c = synth.decode_layer(2, i, 2, device=device, B=B, H=H, T=T, k=k)
            k8, ks = chai.chai_quantize_cache_fp8(c["k_rep"])
            v8, vs = chai.chai_quantize_cache_fp8(c["v"])
            sets.append((c["q"], k8, v8, ks, vs, c["membership"], c["reps"], c["scale"]))
            del c
        ws = chai.new_workspace(int(chai.load().chai_decode_fp8_workspace_bytes(B, H, k, T, D)), device)
        out = torch.empty_like(sets[0][0])

        def step():
            for (q, k8, v8, ks, vs, mem, reps, scale) in sets:
                chai.chai_decode_attention_fp8(q, k8, v8, ks, vs, mem, reps, scale, out=out, workspace=ws)

        for _ in range(warmup):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters):
            step()
        e1.record()
        torch.cuda.synchronize()
        us_eager = e0.elapsed_time(e1) * 1e3 / (iters * len(sets))
        us = graph_time_us(step, len(sets))  # as the main decode number: the calls replayed as one CUDA graph
        nbytes = (k + H) * B * T * D * 1 + (k + H) * B * D * 2 + 4 * B * (H + k) * 2
        gbs = nbytes / (us * 1e-6) / 1e9
        res[f"k{k}"] = {"us_per_layer": us, "us_per_layer_call_by_call": us_eager, "algorithmic_mb": nbytes / 1e6, "gbs": gbs,
                        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                                     "frac": gbs / peaks["hbm"], "peak_source": peaks["source"], "traffic": None}}
        del sets
    # the quantiser on one layer's value cache (read twice: maximum, then conversion; written once in bytes)
    caches = [synth.decode_layer(2, i, 2, device=device, B=B, H=H, T=T, k=8)["v"] for i in range(4)]
    for c in caches[:2]:
        chai.chai_quantize_cache_fp8(c)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for c in caches:
        q8, sc = chai.chai_quantize_cache_fp8(c)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / len(caches)
    qbytes = caches[0].numel() * (2 + 2 + 1)
    res["quantize_v_cache"] = {"us": us, "algorithmic_mb": qbytes / 1e6, "gbs": qbytes / (us * 1e-6) / 1e9,
                               "note": "includes the binding's zero-fill of the byte buffer"}
    res["workload"] = "config2 layer shape (B 16, H 32, T 2048, D 128), e4m3 caches + per-plane scales, bf16 q/out"
    return res


def graph_time_us(run, calls_per_run, reps=4, warmup=3):
    """Mean microseconds per call of `run` (which enqueues `calls_per_run` calls), captured five times into one CUDA
    graph that is replayed `reps` times back to back."""
    for _ in range(warmup):
        run()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(5):
            run()
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * 5 * calls_per_run)


def bench_variants(device, peaks):
    """The method's variants and second shapes: CHAI-QKV decode (values of non-representative heads dropped too: 2k
    cache planes per request) at workload 2's layer shape beside the main decode call timed the same way; CHAI-QKV
    prefill and head_dim-64 prefill at workload 5's shape."""
    w = synth.WORKLOADS[2]
    B, H, T, D, es = w.B, w.H, w.T, w.D, 2
    res = {}
    for k in (8, 16):
        sets = []
        for i in range(8):
            c = synth.decode_layer(2, i, 5, device=device, B=B, H=H, T=T, k=k)
            v_rep = torch.stack([c["v"][b].index_select(0, c["reps"][b].long()) for b in range(B)])
            sets.append((c["q"], c["k_rep"], c["v"], v_rep, c["membership"], c["reps"], c["scale"]))
        ws = chai.new_workspace(max(int(chai.load().chai_decode_qkv_workspace_bytes(B, H, k, T, D, chai.CHAI_BF16)),
                                    chai.chai_decode_workspace_bytes(B, H, k, T, D, chai.CHAI_BF16)), device)
        out = torch.empty_like(sets[0][0])

        def run_qkv():
            for (q, kr, v, vr, mem, reps, scale) in sets:
                chai.chai_decode_attention_qkv(q, kr, vr, mem, reps, scale, out=out, workspace=ws)

        def run_main():
            for (q, kr, v, vr, mem, reps, scale) in sets:
                chai.chai_decode_attention(q, kr, v, mem, reps, scale, out=out, workspace=ws)

        us_q, us_m = graph_time_us(run_qkv, len(sets)), graph_time_us(run_main, len(sets))
        by_q = 2 * k * B * T * D * es + k * B * D * es + H * B * D * es + 4 * B * (H + k)
        by_m = decode_bytes(B, H, k, T, D, es)
        # the main call on as many bytes as the QKV call moves (a shorter context of the same caches): what the same
        # kernel reaches when a launch has this little to stream
        T_eq = max(128, int(round(T * by_q / by_m / 128.0)) * 128)

        def run_main_eq():
            for (q, kr, v, vr, mem, reps, scale) in sets:
                chai.chai_decode_attention(q, kr, v, mem, reps, scale, T=T_eq, out=out, workspace=ws)

        us_e = graph_time_us(run_main_eq, len(sets))
        by_e = decode_bytes(B, H, k, T_eq, D, es)
        res[f"decode_qkv_k{k}"] = {"us": us_q, "algorithmic_mb": by_q / 1e6, "gbs": by_q / us_q / 1e3,
                                   "frac": by_q / us_q / 1e3 / peaks["hbm"],
                                   "main_call_same_timing": {"us": us_m, "algorithmic_mb": by_m / 1e6, "gbs": by_m / us_m / 1e3,
                                                             "frac": by_m / us_m / 1e3 / peaks["hbm"]},
                                   "main_call_on_equal_bytes": {"T": T_eq, "us": us_e, "algorithmic_mb": by_e / 1e6,
                                                                "gbs": by_e / us_e / 1e3, "frac": by_e / us_e / 1e3 / peaks["hbm"]}}
        del sets
        torch.cuda.empty_cache()
    # prefill: CHAI-QKV (one plain head per cluster: k QK^T and k PV products) and head_dim 64 at workload 5's shape
    case = synth.prefill_case(seed=0, device=device)
    Bp, Hp, Tp, Dp, kp = case["B"], case["H"], case["T"], case["D"], case["k"]
    k_rep = chai.chai_compact_k_cache(case["k_full"], case["reps"])
    v_rep = torch.stack([case["v"][b].index_select(0, case["reps"][b].long()) for b in range(Bp)])
    ws = chai.new_workspace(int(chai.load().chai_prefill_qkv_workspace_bytes(Bp, Hp, kp, Tp, Dp, chai.CHAI_BF16)), device)
    out = torch.empty_like(case["q_full"])
    us = graph_time_us(lambda: chai.chai_prefill_attention_qkv(case["q_full"], k_rep, v_rep, case["membership"], case["reps"],
                                                                case["scale"], True, out=out, workspace=ws), 1)
    fl = 2 * Dp * (Tp * (Tp + 1) // 2) * (2 * kp) * Bp
    res["prefill_qkv"] = {"workload": "workload 5's shape, values of the k representatives only", "us": us,
                          "algorithmic_gflop": fl / 1e9, "tflops": fl / us / 1e6, "frac": fl / us / 1e6 / peaks["tf_burst"],
                          "output_mb": out.numel() * 2 / 1e6,
                          "note": "2k contractions per request instead of k + H: the call is bound by writing the H output planes"}
    del case, k_rep, v_rep, out, ws
    g = torch.Generator(device=device).manual_seed(64)
    D64 = 64
    mem, reps = synth.batch_partitions(Bp, Hp, kp, "even", 0, 5, 0)
    mem, reps = torch.as_tensor(mem, device=device), torch.as_tensor(reps, device=device)
    q = (torch.randn((Bp, Hp, Tp, D64), device=device, generator=g) * 0.5).to(torch.bfloat16)
    kr = (torch.randn((Bp, kp, Tp, D64), device=device, generator=g) * 0.5).to(torch.bfloat16)
    v = (torch.randn((Bp, Hp, Tp, D64), device=device, generator=g) * 0.5).to(torch.bfloat16)
    ws = chai.new_workspace(chai.chai_prefill_workspace_bytes(Bp, Hp, kp, Tp, D64, chai.CHAI_BF16), device)
    out = torch.empty_like(q)
    us = graph_time_us(lambda: chai.chai_prefill_attention(q, kr, v, mem, reps, 0.125, True, out=out, workspace=ws), 1)
    fl = prefill_flops(Bp, Hp, kp, Tp, D64)
    res["prefill_head_dim_64"] = {"workload": "B 4, T 2048, H 32, k 8, head_dim 64 (items of four members)", "us": us,
                                  "algorithmic_gflop": fl / 1e9, "tflops": fl / us / 1e6, "frac": fl / us / 1e6 / peaks["tf_burst"]}
    return res


def bench_decode_workload(cfg_id, device, peaks, steps=10, warmup=3):
    """The decode step of another workload, timed like the headline: the step's layer calls captured once in a CUDA
    graph and replayed `steps` times back to back (every layer has its own caches: tens of GB per step)."""
    wl = DecodeWorkload(cfg_id, device)
    for _ in range(warmup):
        wl.step()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        wl.step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(warmup):
        graph.replay()
    ms = time_region(graph.replay, steps, torch.cuda.synchronize) / steps
    ms_eager = time_region(wl.step, steps, torch.cuda.synchronize) / steps
    gbs = wl.bytes_per_step / 1e9 / (ms * 1e-3)
    w = wl.w
    res = {"workload": w.name, "layers": w.layers, "B": w.B, "H": w.H, "T": w.T, "steps": steps,
           "algorithmic_gb_per_step": wl.bytes_per_step / 1e9, "us_per_step": ms * 1e3, "us_per_layer": ms * 1e3 / w.layers,
           "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s", "frac": gbs / peaks["hbm"],
           "eager_us_per_step": ms_eager * 1e3, "launch": "one CUDA graph of the step's layer calls, replayed"}
    del wl, graph
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, choices=[2, 3, 4])
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: keep only the first N layers (not a bench result)")
    ap.add_argument("--skip-extras", action="store_true", help="only the decode step (no prefill/compaction/CPU legs)")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a replayed CUDA graph")
    ap.add_argument("--only", default="", choices=["", "prefill", "compaction", "serving", "fp8", "config1", "workload3", "workload4", "variants"],
                    help="profiling aid: run just this leg and print its object (not the bench line)")
    ap.add_argument("--record-traffic", default="", metavar="NCU_CSV",
                    help="no GPU work: parse an ncu CSV of `--workload W --layers N --skip-extras` into the tracked DRAM-traffic record")
    args = ap.parse_args()
    if args.record_traffic:
        record_traffic(args.record_traffic, args.layers or synth.WORKLOADS[args.workload].layers, args.workload)
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    chai.load()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    ranks = replicas.init_ranks("nccl", device)
    world = ranks.world

    def sync_all():
        torch.cuda.synchronize()
        ranks.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    if args.only:
        leg = {"prefill": bench_prefill, "compaction": bench_compaction, "serving": bench_serving, "fp8": bench_fp8,
               "config1": lambda d, p: bench_config1(d), "variants": bench_variants,
               "workload3": lambda d, p: bench_decode_workload(3, d, p),
               "workload4": lambda d, p: bench_decode_workload(4, d, p)}[args.only]
        print(json.dumps({"leg": args.only, "result": leg(device, peaks)}))
        ranks.close()
        return
    wl = DecodeWorkload(args.workload, device, layers=args.layers)
    w = wl.w
    for _ in range(args.warmup):
        wl.step()
    # The decode step is launch-bound between its 32..64 layer calls, so it is captured once into a CUDA graph
    # and replayed (what a serving loop does); the eager launch loop is timed as well and reported beside it.
    graph = None
    if not args.no_graph:
        try:
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                wl.step()
            torch.cuda.current_stream().wait_stream(side)
            for _ in range(args.warmup):
                graph.replay()
        except Exception as e:  # capture not possible here: time the eager loop only
            print(f"bench.py: CUDA graph capture failed ({e!r}); timing eager launches", file=sys.stderr)
            graph = None
    timed_step = graph.replay if graph is not None else wl.step
    # 1) device-resident timing: exactly K steps, two events
    with ClockSampler(local_rank) as clk:
        ms_total = time_region(timed_step, args.steps, sync_all)
        ms_eager = time_region(wl.step, args.steps, sync_all) if graph is not None else ms_total
        # the same K steps with an event after every step: median and best step beside the mean
        step_ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        sync_all()
        step_ev[0].record()
        for s_i in range(args.steps):
            timed_step()
            step_ev[s_i + 1].record()
        torch.cuda.synchronize()
        step_ms = [step_ev[i].elapsed_time(step_ev[i + 1]) for i in range(args.steps)]
        # 2) same K steps again with an event after every layer call: per-launch durations for the roofline
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(w.layers + 1)] for _ in range(args.steps)]
        sync_all()
        for s in range(args.steps):
            wl.step_with_events(events[s])
        torch.cuda.synchronize()
    layer_ms = np.array([[ev[i].elapsed_time(ev[i + 1]) for i in range(w.layers)] for ev in events])
    # 3) end to end through the host-buffer entry point: H2D of every layer's queries, D2H of every output
    wl.make_host_buffers()
    for _ in range(3):
        wl.step_host()
    ms_e2e = time_region(wl.step_host, args.steps, sync_all)
    ms_e2e_blocking = time_region(wl.step_host_blocking, args.steps, sync_all)
    wl.make_pipeline()
    for _ in range(3):
        wl.step_host_pipelined()
    ms_e2e_pipe = time_region(wl.step_host_pipelined, args.steps, sync_all)

    ms_total, ms_e2e, ms_eager, ms_e2e_blocking, ms_e2e_pipe = ranks.max_over_ranks(
        [ms_total, ms_e2e, ms_eager, ms_e2e_blocking, ms_e2e_pipe])
    ms_step = ms_total / args.steps
    value = replicas.whole_job_throughput(ranks, wl.bytes_per_step / 1e9, ms_step * 1e-3)["value"]
    e2e_value = replicas.whole_job_throughput(ranks, wl.bytes_per_step / 1e9, ms_e2e / args.steps * 1e-3)["value"]

    if rank == 0:
        traffic_ratio, traffic_rec = load_traffic_ratio()
        # average launch duration over the timed region itself (K steps x layers launches, gaps included)
        per_launch_ms = ms_step / w.layers
        achieved = float(np.mean(wl.bytes_per_layer)) / (per_launch_ms * 1e-3) / 1e9
        eager_value = wl.bytes_per_step / 1e9 / (ms_eager / args.steps * 1e-3) * world
        by_k = {}
        for c, col in zip(wl.layers, layer_ms.T):
            by_k.setdefault(c["k"], []).append(float(np.median(col)) * 1e3)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "us_per_step": ms_step * 1e3,
            "us_per_step_median": statistics.median(step_ms) * 1e3, "us_per_step_best": min(step_ms) * 1e3,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name + (" (TRUNCATED for profiling)" if args.layers else ""), "layers": w.layers, "B": w.B, "H": w.H, "D": w.D, "T": w.T,
                       "k_per_layer": [c["k"] for c in wl.layers], "partition": w.partition,
                       "algorithmic_gb_per_step": wl.bytes_per_step / 1e9,
                       "arithmetic": "bf16 caches, queries and outputs; fp32 scores, softmax and accumulation",
                       "l2": "inputs larger than L2: every layer has its own >=168 MiB caches, 12+ GB per step",
                       "launch": ("one CUDA graph of the step's layer calls, replayed" if graph is not None else "eager launches"),
                       "multi_gpu": "independent replicas, no data-path collective"},
            "eager": {"value": eager_value, "unit": UNIT, "ms_per_step": ms_eager / args.steps,
                      "note": "the same K steps launched call by call from the host"},
            "gpu_launches": wl.launches_per_step * args.steps,
            "roofline": {"bound": "hbm", "kernel": "decode_persistent_kernel (one launch per layer call)",
                         "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                         "peak_source": peaks["source"],
                         # DRAM read+write bytes per launch: the ratio to the algorithmic bytes that an ncu capture of
                         # this kernel measured (the tracked record names the capture), applied to the mean launch
                         # here; null when there is no record
                         "traffic": (traffic_ratio * float(np.mean(wl.bytes_per_layer)) if traffic_ratio else None),
                         "traffic_unit": "bytes per launch",
                         "traffic_source": (None if traffic_rec is None else
                                            {"ratio_to_algorithmic": traffic_ratio, "measured_on": traffic_rec["workload"],
                                             "launches": traffic_rec["launches_captured"],
                                             "note": "ncu dram__bytes_read.sum + dram__bytes_write.sum per launch, scaled by the units processed"}),
                         "us_per_layer_by_k": {str(k): statistics.median(v) for k, v in sorted(by_k.items())},
                         "us_per_layer_by_k_note": "eager launches with an event after every layer call",
                         "frac_of_nominal_8TBs": achieved / 8000.0},
            "e2e": {"value": replicas.whole_job_throughput(ranks, wl.bytes_per_step / 1e9,
                                                           ms_e2e_pipe / args.steps * 1e-3)["value"],
                    "unit": UNIT, "us_per_step": ms_e2e_pipe / args.steps * 1e3,
                    "h2d_bytes_per_step": w.layers * w.B * w.H * w.D * wl.es,
                    "d2h_bytes_per_step": w.layers * w.B * w.H * w.D * wl.es,
                    "note": "chai_decode_attention_host_streams per layer: queries from pinned host memory, outputs back "
                            "to it, upload / kernels / download on three streams, a staging buffer per layer, one wait "
                            "per step; caches stay resident",
                    "one_stream": {"value": e2e_value, "us_per_step": ms_e2e / args.steps * 1e3,
                                   "note": "chai_decode_attention_host_async: everything on one stream, one wait per step"},
                    "blocking_per_layer": {
                        "value": replicas.whole_job_throughput(ranks, wl.bytes_per_step / 1e9,
                                                               ms_e2e_blocking / args.steps * 1e-3)["value"],
                        "us_per_step": ms_e2e_blocking / args.steps * 1e3,
                        "note": "chai_decode_attention_host: the host waits after every layer call"}},
            "clocks": clk.summary(),
        }
        if not args.skip_extras and world == 1:
            del wl
            torch.cuda.empty_cache()
            line["prefill"] = bench_prefill(device, peaks)
            line["compaction"] = bench_compaction(device, peaks)
            line["serving"] = bench_serving(device, peaks)
            line["fp8_decode"] = bench_fp8(device, peaks)
            line["config1"] = bench_config1(device)
            line["variants"] = bench_variants(device, peaks)
            others = {f"workload{c}": bench_decode_workload(c, device, peaks) for c in (3, 4) if c != args.workload}
            line["decode_other_workloads"] = others
            # Compact summaries of the other legs inside the roofline object, so that this one object carries the
            # whole metric: decode at every model-shaped workload, prefill, compaction, the serving and fp8 steps.
            rl = line["roofline"]
            rl[f"workload{args.workload}"] = {"us_per_step": ms_step * 1e3, "achieved": achieved, "frac": achieved / peaks["hbm"]}
            for name, o in others.items():
                rl[name] = {k2: o[k2] for k2 in ("us_per_step", "us_per_layer", "achieved", "frac", "algorithmic_gb_per_step")}
            pf = line["prefill"]
            rl["prefill"] = {"workload": pf["workload"], "us": pf["ms_attention"] * 1e3, "achieved": pf["tflops"],
                             "peak": peaks["tf_burst"], "unit": "TFLOP/s", "frac": pf["roofline"]["frac"], "peak_kind": "burst",
                             "algorithmic_gflop": pf["algorithmic_gflop"], "bound": "tensor",
                             "sustained_frac": pf["sustained"]["frac"],
                             "longer_prompts_frac": {k2: v2["frac_of_burst_peak"] for k2, v2 in pf["longer_prompts"].items()}}
            rl["compaction"] = {k2: {"us": v2["us"], "achieved": v2["gbs"], "frac": v2["frac"]}
                                for k2, v2 in line["compaction"]["by_k"].items()}
            sv = line["serving"]
            rl["ragged_decode"] = {"us": sv["ragged_decode"]["back_to_back"]["us"], "achieved": sv["ragged_decode"]["back_to_back"]["gbs"],
                                   "frac": sv["ragged_decode"]["back_to_back"]["frac"], "timing": "back to back over four cache sets, graph replay",
                                   "single_cold_call": {"us": sv["ragged_decode"]["us"], "frac": sv["ragged_decode"]["roofline"]["frac"]},
                                   "us_over_full_length_us_times_byte_ratio": sv["ragged_decode"]["back_to_back"]["us_over_full_length_us_times_byte_ratio"]}
            rl["fp8_decode"] = {k2: {"us_per_layer": line["fp8_decode"][k2]["us_per_layer"], "achieved": line["fp8_decode"][k2]["gbs"],
                                     "frac": line["fp8_decode"][k2]["roofline"]["frac"]} for k2 in ("k8", "k32")}
            vr = line["variants"]
            rl["variants"] = {"decode_qkv_k8": {k2: vr["decode_qkv_k8"][k2] for k2 in ("us", "gbs", "frac")},
                              "decode_qkv_k16": {k2: vr["decode_qkv_k16"][k2] for k2 in ("us", "gbs", "frac")},
                              "prefill_qkv": {k2: vr["prefill_qkv"][k2] for k2 in ("us", "tflops", "frac")},
                              "prefill_head_dim_64": {k2: vr["prefill_head_dim_64"][k2] for k2 in ("us", "tflops", "frac")}}
            line["cpu_baseline"] = cpu_baseline_decode(args.workload, 0)
            line["cpu_baseline"]["prefill"] = cpu_baseline_prefill()
        print(json.dumps(line))
    ranks.close()


if __name__ == "__main__":
    main()

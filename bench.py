#!/usr/bin/env python
"""Benchmark of the JetViT token mixers on B200.

One "step" is one pass of the whole hot path at the DINOv3-L high-resolution
shape (B=8, heads=16, 64x64 token grid, head_dim 64, bf16): jv_hybrid_mixers with
schedule "LWF" over three layers of fresh synthetic Q/K/V -- the linear-attention
block (with its squeeze dynamic convolution), 16x16 window attention and full
attention.  `value` is mixer tokens/s (layers x B x N per step) with inputs
resident in HBM; `e2e` is the same step with host buffers (pinned), host<->device
copies inside the timed region.  Each mixer is also timed on its own (tokens/s,
achieved GB/s or TFLOP/s against the measured peaks), and the 24-layer 128x128
hybrid stack is timed against the same stack run all-F.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Under torchrun (N > 1) every rank runs the same per-GPU workload on its own GPU
(the path shards over independent (batch, head) units: no data-path collective).
`--impl reference` times the float64 CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_26636_b200 import inputs

METRIC = "mixer tokens/sec (L+W+F stack at ViT-L shapes)"
UNIT = "tokens/s"
STEP_SCHEDULE = "LWF"
WIN = 16
# DRAM traffic of the dominant kernel comes from an ncu capture; the record of that capture names the
# kernel's source files and their hash, and the figure is reported only while the hash still matches
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "attn_f4_kernel_dinov3_l.traffic.json")


TRAFFIC_SOURCES = ["paper_2605_26636_b200/csrc/attn_f4.cu", "paper_2605_26636_b200/csrc/tc_common.cuh"]


def record_traffic(csv_path):
    """Writes TRAFFIC_RECORD from `ncu -i <report> --page raw --csv` output of a capture of attn_f4_kernel
    (`ncu --set full ... python bench.py --single F`): DRAM bytes per launch and the hash of the kernel's source."""
    import csv
    import hashlib
    rows = list(csv.reader(open(csv_path)))
    hdr, units = rows[0], rows[1]
    ix = {h: i for i, h in enumerate(hdr)}
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    vals = []
    for r in rows[2:]:
        if "attn_f4_kernel" not in r[ix["Kernel Name"]]:
            continue
        tot = 0.0
        for key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            tot += float(r[ix[key]].replace(",", "")) * scale[units[ix[key]]]
        vals.append(tot)
    if not vals:
        raise SystemExit("no attn_f4_kernel launch in " + csv_path)
    h = hashlib.sha256()
    for rel in TRAFFIC_SOURCES:
        h.update(open(os.path.join(ROOT, rel), "rb").read())
    rec = {"kernel": "attn_f4_kernel", "workload": "F at dinov3_l (B=8, H=16, N=4096, D=64, bf16)", "launches": len(vals),
           "dram_bytes_per_launch": int(sum(vals) / len(vals)), "sources": TRAFFIC_SOURCES, "sha256": h.hexdigest(),
           "how": "ncu --set full --clock-control none -k regex:attn_f4 python bench.py --single F --steps 2 --warmup 1; "
                  "ncu -i <report> --page raw --csv; python bench.py --record-traffic <csv>"}
    json.dump(rec, open(TRAFFIC_RECORD, "w"), indent=1)
    print(json.dumps(rec))


def measured_traffic():
    """(bytes per launch or None, note): dram__bytes_read.sum + dram__bytes_write.sum of one launch of the
    dominant kernel, valid only for the source it was captured from."""
    import hashlib
    try:
        rec = json.load(open(TRAFFIC_RECORD))
        h = hashlib.sha256()
        for rel in rec["sources"]:
            h.update(open(os.path.join(ROOT, rel), "rb").read())
        if h.hexdigest() == rec["sha256"]:
            return int(rec["dram_bytes_per_launch"]), "ncu capture of the current source"
        return None, "the kernel's source has changed since the ncu capture"
    except (OSError, KeyError, ValueError):
        return None, "no ncu record"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- algorithmic work
def alg_bytes(B, H, N, D, esz=2, dwc=False):
    """Q, K, V read once, O written once (V read twice with the convolution)."""
    return B * H * N * D * esz * (5 if dwc else 4)


def alg_flops_attn(B, H, Hg, Wg, D, wh, ww, prefix=0):
    """2 flops per MAC over valid (query, key) pairs only, QK^T and PV; with prefix tokens every
    window token also attends them, and they attend everything."""
    pairs = prefix * (prefix + Hg * Wg)
    for y0 in range(0, Hg, wh):
        for x0 in range(0, Wg, ww):
            n = min(wh, Hg - y0) * min(ww, Wg - x0)
            pairs += n * (n + prefix)
    return 4 * D * pairs * B * H


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            f = [x.strip() for x in s.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx = max(mx, float(f[1]))
            except ValueError:
                continue
            for n, val in zip(names, f[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- timing helpers
def time_calls(fn, steps, warmup, stream):
    """Device time per call (ms): CUDA events on the launching stream around `steps` calls."""
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        fn(warmup + i)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(x: float, world: int, device=None) -> float:
    """MAX all-reduce of a per-rank time (the step time of a multi-GPU run is the slowest rank's)."""
    if world <= 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_layer_ids(rank: int, n_layers: int):
    """Layer indices that seed rank `rank`'s inputs: every rank draws its own shard (the path shards
    over independent (batch, head) units, so ranks share nothing but the timing barrier)."""
    return [100 * rank + l for l in range(n_layers)]


# ----------------------------------------------------------------------------- oracle legs
def oracle_sample_step(w, scale=1.0):
    """A bounded sample of one step for the CPU oracle (about 10 s on 16 cores, 30 s on 8,
    at scale 1): L with the dynamic convolution and W on ceil(scale * B) batch samples,
    F on all query rows of round(scale * B * H) of the B*H (batch, head) pairs; each
    mixer's time is extrapolated to the whole step by its sampled fraction.
    Returns (seconds spent, extrapolated seconds of a whole step, description,
    threads used)."""
    from oracle import jv_oracle
    C = w.H * w.D
    d = inputs.dwc_weights(C, C // 8, 3, inputs.seed_for(w.cfg, 0, 3))
    nB = max(1, min(w.B, int(np.ceil(scale * w.B))))
    q, k, v = inputs.qkv(w, layer=0, shape=(nB, w.H, w.N, w.D))
    t0 = time.perf_counter()
    jv_oracle.linear_attn(q, k, v, w.Hg, w.Wg, dwc=d)
    tL = time.perf_counter() - t0
    q, k, v = inputs.qkv(w, layer=1, shape=(nB, w.H, w.N, w.D))
    t0 = time.perf_counter()
    jv_oracle.window_attn(q, k, v, w.Hg, w.Wg, WIN, WIN)
    tW = time.perf_counter() - t0
    nF = max(1, min(w.B * w.H, int(round(w.B * w.H * scale))))
    q, k, v = inputs.qkv(w, layer=2, shape=(1, nF, w.N, w.D))
    t0 = time.perf_counter()
    jv_oracle.full_attn(q, k, v)
    tF = time.perf_counter() - t0
    full_step_s = (tL + tW) * w.B / nB + tF * (w.B * w.H) / nF
    desc = (f"L+DWC on {nB}/{w.B} of the batch ({tL:.2f}s), W on {nB}/{w.B} of the batch ({tW:.2f}s), "
            f"F on {nF} of {w.B * w.H} (batch, head) pairs ({tF:.2f}s); each extrapolated by its fraction")
    return tL + tW + tF, full_step_s, desc, jv_oracle.num_threads()


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    w = inputs.WORKLOADS["dinov3_l"]
    step_tokens = len(STEP_SCHEDULE) * w.tokens
    # size the per-step sample so that the whole run stays near two minutes
    n_warm = min(args.warmup, 1)
    scale = min(1.0, 120.0 / (30.0 * (args.steps + n_warm)))
    for _ in range(n_warm):
        oracle_sample_step(w, scale)
    spent, full = [], []
    for _ in range(args.steps):
        s, f, desc, cores = oracle_sample_step(w, scale)
        spent.append(s)
        full.append(f)
    step_s = float(np.mean(full))
    value = step_tokens / step_s
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "extrapolated": True,
            "extrapolated_note": "each step times a bounded sample of the workload; ms_per_step and value scale every mixer's "
                                 "time by its sampled fraction",
            "config": {"workload": "dinov3_l 64x64 grid B=8 H=16 D=64, schedule LWF (CPU oracle, sampled)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- CUDA arm
def run_cuda(args):
    from paper_2605_26636_b200 import jetvit as jv
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    jv.lib()
    peaks = load_peaks()
    stream = torch.cuda.current_stream()
    w = inputs.WORKLOADS["dinov3_l"]
    nL = len(STEP_SCHEDULE)
    C = w.H * w.D

    # ---- inputs: three layers of Q/K/V in pinned host memory and on the device
    host = [[t.pin_memory() for t in inputs.qkv(w, layer=lid)] for lid in rank_layer_ids(rank, nL)]
    dq, dk, dv = ([host[l][i].to(dev, non_blocking=True) for l in range(nL)] for i in range(3))
    outs = [torch.empty_like(t) for t in dq]
    host_out = [torch.empty(w.shape, dtype=torch.bfloat16).pin_memory() for _ in range(nL)]
    dwc_host = inputs.dwc_weights(C, C // 8, 3, inputs.seed_for(w.cfg, 0, 3))
    dwc_dev = {k: (v.to(dev) if hasattr(v, "to") else v) for k, v in dwc_host.items()}
    dwcs = [dwc_dev if m == "L" else None for m in STEP_SCHEDULE]
    shape = jv.make_shape(dq[0], w.Hg, w.Wg)
    ws = jv.alloc_workspace("S", shape, jv.make_dwc(dwc_dev, dev), dev)
    torch.cuda.synchronize()

    # One step = the schedule driver over the three layers.  It is issued as one jv_hybrid_mixers
    # call per layer so that events between the calls give each mixer's time inside the timed region.
    def step(_i=0, ev=None):
        for l, m in enumerate(STEP_SCHEDULE):
            if ev is not None:
                ev[l].record(stream)
            jv.hybrid_mixers(m, dq[l:l + 1], dk[l:l + 1], dv[l:l + 1], w.Hg, w.Wg, WIN, WIN, dwc=dwcs[l:l + 1],
                             out=outs[l:l + 1], ws=ws)
        if ev is not None:
            ev[nL].record(stream)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the timed region: exactly K steps between barrier + synchronize
    for i in range(args.warmup):
        step()
    barrier()
    l0 = jv.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_ev = min(args.steps, 64)            # steps whose per-layer events are kept
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(nL + 1)] for _ in range(n_ev)]
    with ClockSampler(local) as clk:
        e0.record(stream)
        for i in range(args.steps):
            step(i, evs[i] if i < n_ev else None)
        e1.record(stream)
        barrier()
    launches = jv.launch_count() - l0
    ms = e0.elapsed_time(e1) / args.steps
    layer_ms = [float(np.mean([evs[i][l].elapsed_time(evs[i][l + 1]) for i in range(n_ev)])) for l in range(nL)]
    ms = max_over_ranks(ms, world, dev)
    assert jv.device_status() == jv.JV_OK, "a kernel reported a timeout"
    step_tokens = nL * w.tokens
    value = world * step_tokens / (ms * 1e-3)

    # ---- the same step for at least a second: what the clocks settle at under the power cap
    n_sus = max(50, int(1.2e3 / max(ms, 1e-3)))
    with ClockSampler(local) as clk_sus:
        e0.record(stream)
        for i in range(n_sus):
            step()
        e1.record(stream)
        barrier()
    ms_sus = max_over_ranks(e0.elapsed_time(e1) / n_sus, world, dev)
    cs = clk_sus.summary()
    sustained = {"steps": n_sus, "ms_per_step": ms_sus, "value": world * step_tokens / (ms_sus * 1e-3), "unit": UNIT,
                 "clocks": cs, "ms_x_mhz": (ms_sus * cs["sm_mhz"]) if cs.get("sm_mhz") else None,
                 "burst_ms_x_mhz": None}   # filled in below, once the burst region's clock summary exists

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region.
    # The way a user would drive the library from host data: three streams (upload, mixers, download)
    # and two sets of device buffers, so that step i + 1 uploads while step i computes and step i - 1
    # downloads.  Every step still moves all its inputs in from pinned host memory and all its outputs back.
    sets = [(dq, dk, dv, outs),
            tuple([torch.empty_like(t) for t in lst] for lst in (dq, dk, dv, outs))]
    s_up, s_down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_done = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    torch.cuda.synchronize()
    for b in range(2):
        ev_done[b].record(stream)
        ev_out[b].record(stream)

    def e2e_step(i):
        b = i & 1
        q_, k_, v_, o_ = sets[b]
        with torch.cuda.stream(s_up):
            s_up.wait_event(ev_done[b])           # the mixers of step i - 2 have read this input set
            for l in range(nL):
                for j, dst in enumerate((q_, k_, v_)):
                    dst[l].copy_(host[l][j], non_blocking=True)
            ev_in[b].record(s_up)
        stream.wait_event(ev_in[b])
        stream.wait_event(ev_out[b])              # step i - 2's outputs have been downloaded
        for l, m in enumerate(STEP_SCHEDULE):
            jv.hybrid_mixers(m, q_[l:l + 1], k_[l:l + 1], v_[l:l + 1], w.Hg, w.Wg, WIN, WIN, dwc=dwcs[l:l + 1],
                             out=o_[l:l + 1], ws=ws)
        ev_done[b].record(stream)
        with torch.cuda.stream(s_down):
            s_down.wait_event(ev_done[b])
            for l in range(nL):
                host_out[l].copy_(o_[l], non_blocking=True)
            ev_out[b].record(s_down)

    n_e2e = max(4, min(args.steps, 8))
    for i in range(2):
        e2e_step(i)
    barrier()
    e0.record(s_up)
    for i in range(n_e2e):
        e2e_step(i)
    e1.record(s_down)
    barrier()
    ms_e2e = e0.elapsed_time(e1) / n_e2e
    ms_e2e = max_over_ranks(ms_e2e, world, dev)
    tensor_bytes = int(np.prod(w.shape)) * 2
    e2e = {"value": world * step_tokens / (ms_e2e * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e,
           "h2d_bytes_per_step": 3 * nL * tensor_bytes, "d2h_bytes_per_step": nL * tensor_bytes,
           "how": "pinned host buffers; upload, mixers and download on three streams, two device buffer sets"}

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- per-mixer timings (rank 0; rotating over the three layers' tensors: 805 MB > L2)
    per = {}
    K, W = min(max(args.steps, 10), 100), max(min(args.warmup, 10), 3)
    hbm, tf = peaks["hbm_gbs"], peaks["bf16_tflops"]

    def add(name, fn, bytes_, flops, bound):
        t_ms = time_calls(fn, K, W, stream)
        gbs, tfl = bytes_ / t_ms / 1e6, flops / t_ms / 1e9
        per[name] = {"ms": t_ms, "tokens_per_s": w.tokens / (t_ms * 1e-3), "GBps": gbs, "TFLOPs": tfl,
                     "frac_hbm": gbs / hbm, "frac_tensor": tfl / tf, "bound": bound}

    r = lambda i: i % nL
    add("L", lambda i: jv.linear_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, out=outs[r(i)], ws=ws),
        alg_bytes(*w.shape), 0.0, "hbm")
    add("L+dwc", lambda i: jv.linear_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, dwc=dwc_dev, out=outs[r(i)], ws=ws),
        alg_bytes(*w.shape, dwc=True), 0.0, "hbm")
    add("W", lambda i: jv.window_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, WIN, WIN, out=outs[r(i)]),
        alg_bytes(*w.shape), alg_flops_attn(w.B, w.H, w.Hg, w.Wg, w.D, WIN, WIN), "hbm")
    f_flops = alg_flops_attn(w.B, w.H, w.Hg, w.Wg, w.D, w.Hg, w.Wg)
    add("F", lambda i: jv.full_attn(dq[r(i)], dk[r(i)], dv[r(i)], out=outs[r(i)]),
        alg_bytes(*w.shape), f_flops, "tensor")

    # Table 1's variants of the linear block at mixer level, same shape, same inputs: ReLU linear attention,
    # + static DWC, + DWC + focusing factor (p = 3), + token-wise dynamic DWC, + squeeze dynamic DWC
    dwc_static = {"k": 3, "R": 0, "b2": dwc_dev["b2"]}
    dwc_token = dict(dwc_dev, token_wise=1)
    shape_l = jv.make_shape(dq[0], w.Hg, w.Wg)
    ws_f = jv.alloc_workspace("f", shape_l, jv.make_dwc(dwc_static, dev), dev)
    ws_t = jv.alloc_workspace("L", shape_l, jv.make_dwc(dwc_token, dev), dev)
    table1 = {}
    for name, fn in (
            ("relu_la", lambda i: jv.linear_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, out=outs[r(i)], ws=ws)),
            ("static_dwc", lambda i: jv.linear_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, dwc=dwc_static, out=outs[r(i)], ws=ws)),
            ("static_dwc_focus_p3", lambda i: jv.linear_attn_focused(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, 3.0, dwc=dwc_static,
                                                                     out=outs[r(i)], ws=ws_f)),
            ("tokenwise_dyn_dwc", lambda i: jv.linear_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, dwc=dwc_token, out=outs[r(i)], ws=ws_t)),
            ("squeeze_dyn_dwc", lambda i: jv.linear_attn(dq[r(i)], dk[r(i)], dv[r(i)], w.Hg, w.Wg, dwc=dwc_dev, out=outs[r(i)], ws=ws))):
        t_ms = time_calls(fn, min(K, 30), 3, stream)
        table1[name] = {"ms": t_ms, "tokens_per_s": w.tokens / (t_ms * 1e-3)}
    table1["note"] = ("mixer-level times of the rows of the paper's Table 1 (whole-model H100 latencies there: 5.33 / 5.72 / 6.00 / "
                      "8.94 / 5.88 ms); only the ordering is comparable")
    del ws_f, ws_t

    # the projections either side of a mixer (outside the step: the metric counts mixers only)
    Cm = w.H * w.D
    px = inputs.normal((w.B, w.N, Cm), inputs.seed_for(w.cfg, 0, 5), "bf16").to(dev)
    pw, pb = (t.to(dev) for t in inputs.proj_weights(3 * Cm, Cm, inputs.seed_for(w.cfg, 0, 6)))
    pwo, pbo = (t.to(dev) for t in inputs.proj_weights(Cm, Cm, inputs.seed_for(w.cfg, 0, 7)))
    py = torch.empty_like(px)
    tok = w.B * w.N
    add("qkv_proj", lambda i: jv.qkv_proj(px, pw, pb, w.H, w.Hg, w.Wg, out=tuple(outs)),
        2 * (tok * Cm + 3 * Cm * Cm + 3 * tok * Cm), 2.0 * tok * 3 * Cm * Cm, "tensor")
    add("out_proj", lambda i: jv.out_proj(outs[r(i)], pwo, pbo, w.Hg, w.Wg, out=py),
        2 * (2 * tok * Cm + Cm * Cm), 2.0 * tok * Cm * Cm, "tensor")
    del px, py

    # the same shape with the five prefix tokens of DINOv3 (class token + four registers) in front of the grid
    P5 = 5
    pq = [[t.to(dev) for t in inputs.custom_qkv(w.B, w.H, P5 + w.N, w.D, "bf16", seed=4100 + l)] for l in range(3)]
    po = [torch.empty_like(pq[0][0]) for _ in range(3)]
    tokp = w.B * (P5 + w.N)

    def addp(name, fn, bytes_, flops, bound):
        t_ms = time_calls(fn, K, W, stream)
        per[name] = {"ms": t_ms, "tokens_per_s": tokp / (t_ms * 1e-3), "GBps": bytes_ / t_ms / 1e6, "TFLOPs": flops / t_ms / 1e9,
                     "frac_hbm": bytes_ / t_ms / 1e6 / hbm, "frac_tensor": flops / t_ms / 1e9 / tf, "bound": bound}
    bp = alg_bytes(w.B, w.H, P5 + w.N, w.D)
    addp("L+dwc@prefix5", lambda i: jv.linear_attn(*pq[r(i)], w.Hg, w.Wg, dwc=dwc_dev, out=po[r(i)], ws=ws, prefix=P5),
         alg_bytes(w.B, w.H, P5 + w.N, w.D, dwc=True), 0.0, "hbm")
    addp("W@prefix5", lambda i: jv.window_attn(*pq[r(i)], w.Hg, w.Wg, WIN, WIN, out=po[r(i)], prefix=P5), bp,
         alg_flops_attn(w.B, w.H, w.Hg, w.Wg, w.D, WIN, WIN, prefix=P5), "hbm")
    del pq, po

    # the same shape with q, k, v as slices of a fused [B, N, 3, H, D] activation (token stride 3 H D), the form in
    # which a model's QKV projection leaves them; the mixers read them in place through strided tensor maps
    fq = []
    for l in range(3):
        qkv3 = torch.stack([t.permute(0, 2, 1, 3) for t in (dq[l], dk[l], dv[l])], dim=2).contiguous()
        fq.append((qkv3, [qkv3[:, :, i].permute(0, 2, 1, 3) for i in range(3)]))
    add("L+dwc@fused_qkv", lambda i: jv.linear_attn(*fq[r(i)][1], w.Hg, w.Wg, dwc=dwc_dev, out=outs[r(i)], ws=ws),
        alg_bytes(*w.shape, dwc=True), 0.0, "hbm")
    add("W@fused_qkv", lambda i: jv.window_attn(*fq[r(i)][1], w.Hg, w.Wg, WIN, WIN, out=outs[r(i)]),
        alg_bytes(*w.shape), alg_flops_attn(w.B, w.H, w.Hg, w.Wg, w.D, WIN, WIN), "hbm")
    add("F@fused_qkv", lambda i: jv.full_attn(*fq[r(i)][1], out=outs[r(i)]),
        alg_bytes(*w.shape), f_flops, "tensor")
    del fq

    # other model sizes at the 1024 x 2048 image of Tables 1 and 3 (64 x 128 token grid): 12 heads (ViT-B), 24 heads (Giant)
    for tag, heads in (("vitb_64x128", 12), ("giant_64x128", 24)):
        Bx, Hgx, Wgx = 4, 64, 128
        xq = [[t.to(dev) for t in inputs.custom_qkv(Bx, heads, Hgx * Wgx, 64, "bf16", seed=8000 + heads + l)] for l in range(2)]
        xo = [torch.empty_like(xq[0][0]) for _ in range(2)]
        Cx = heads * 64
        dx = {kk: (vv.to(dev) if hasattr(vv, "to") else vv) for kk, vv in inputs.dwc_weights(Cx, Cx // 8, 3, 8100 + heads).items()}
        wsx = jv.alloc_workspace("L", jv.make_shape(xq[0][0], Hgx, Wgx), jv.make_dwc(dx, dev), dev)
        rows = {"L+dwc": (lambda i: jv.linear_attn(*xq[i % 2], Hgx, Wgx, dwc=dx, out=xo[i % 2], ws=wsx),
                          alg_bytes(Bx, heads, Hgx * Wgx, 64, dwc=True), 0.0, "hbm"),
                "W": (lambda i: jv.window_attn(*xq[i % 2], Hgx, Wgx, WIN, WIN, out=xo[i % 2]),
                      alg_bytes(Bx, heads, Hgx * Wgx, 64), alg_flops_attn(Bx, heads, Hgx, Wgx, 64, WIN, WIN), "hbm"),
                "F": (lambda i: jv.full_attn(*xq[i % 2], out=xo[i % 2]),
                      alg_bytes(Bx, heads, Hgx * Wgx, 64), alg_flops_attn(Bx, heads, Hgx, Wgx, 64, Hgx, Wgx), "tensor")}
        for name, (fn, bytes_, flops, bound) in rows.items():
            Kx = 5 if name == "F" else K
            t_ms = time_calls(fn, Kx, 3, stream)
            per[f"{name}@{tag}"] = {"ms": t_ms, "tokens_per_s": Bx * Hgx * Wgx / (t_ms * 1e-3), "GBps": bytes_ / t_ms / 1e6,
                                    "TFLOPs": flops / t_ms / 1e9, "frac_hbm": bytes_ / t_ms / 1e6 / hbm,
                                    "frac_tensor": flops / t_ms / 1e9 / tf, "bound": bound}
        del xq, xo, wsx

    # head_dim 128 (a 7B-class model: 32 heads of 128 channels; here 8 of them, B = 8, 64 x 64 grid): F on its own kernel
    dq8 = [[t.to(dev) for t in inputs.custom_qkv(8, 8, w.N, 128, "bf16", seed=8300 + l)] for l in range(3)]
    do8 = [torch.empty_like(dq8[0][0]) for _ in range(3)]
    t_ms = time_calls(lambda i: jv.full_attn(*dq8[r(i)], out=do8[r(i)]), min(K, 50), 3, stream)
    fl8 = 4.0 * 8 * 8 * w.N * w.N * 128
    by8 = alg_bytes(8, 8, w.N, 128)
    per["F@d128_64x64"] = {"ms": t_ms, "tokens_per_s": 8 * w.N / (t_ms * 1e-3), "GBps": by8 / t_ms / 1e6, "TFLOPs": fl8 / t_ms / 1e9,
                           "frac_hbm": by8 / t_ms / 1e6 / hbm, "frac_tensor": fl8 / t_ms / 1e9 / tf, "bound": "tensor"}
    t_ms = time_calls(lambda i: jv.window_attn(*dq8[r(i)], w.Hg, w.Wg, WIN, WIN, out=do8[r(i)]), K, W, stream)
    fw8 = alg_flops_attn(8, 8, w.Hg, w.Wg, 128, WIN, WIN)
    per["W@d128_64x64"] = {"ms": t_ms, "tokens_per_s": 8 * w.N / (t_ms * 1e-3), "GBps": by8 / t_ms / 1e6, "TFLOPs": fw8 / t_ms / 1e9,
                           "frac_hbm": by8 / t_ms / 1e6 / hbm, "frac_tensor": fw8 / t_ms / 1e9 / tf, "bound": "hbm"}
    del dq8, do8

    # ragged DepthAnythingV2-L grid (73x73, B=4): F and W with masked edge windows
    w4 = inputs.WORKLOADS["dav2_l"]
    q4 = [[t.to(dev) for t in inputs.qkv(w4, layer=l)] for l in range(3)]
    o4 = [torch.empty_like(q4[0][0]) for _ in range(3)]

    def add4(name, fn, bytes_, flops, bound):
        t_ms = time_calls(fn, K, W, stream)
        per[name] = {"ms": t_ms, "tokens_per_s": w4.tokens / (t_ms * 1e-3), "GBps": bytes_ / t_ms / 1e6,
                     "TFLOPs": flops / t_ms / 1e9, "frac_hbm": bytes_ / t_ms / 1e6 / hbm,
                     "frac_tensor": flops / t_ms / 1e9 / tf, "bound": bound}
    add4("F@dav2_73x73", lambda i: jv.full_attn(*q4[r(i)], out=o4[r(i)]),
         alg_bytes(*w4.shape), alg_flops_attn(w4.B, w4.H, w4.Hg, w4.Wg, w4.D, w4.Hg, w4.Wg), "tensor")
    add4("W@dav2_73x73", lambda i: jv.window_attn(*q4[r(i)], w4.Hg, w4.Wg, WIN, WIN, out=o4[r(i)]),
         alg_bytes(*w4.shape), alg_flops_attn(w4.B, w4.H, w4.Hg, w4.Wg, w4.D, WIN, WIN), "hbm")
    del q4, o4

    # 24-layer hybrid stack at 128x128 against the same stack run all-F
    w5 = inputs.WORKLOADS["hybrid24"]
    base = [t.to(dev) for t in inputs.qkv(w5, layer=0)]
    q5 = [[torch.roll(t, l, dims=2) if l else t for t in base] for l in range(4)]   # 4 distinct layer inputs
    lq, lk, lv = ([q5[l % 4][i] for l in range(w5.n_layers)] for i in range(3))
    lo = [torch.empty_like(base[0]) for _ in range(4)]
    louts = [lo[l % 4] for l in range(w5.n_layers)]
    ws5 = jv.alloc_workspace("S", jv.make_shape(base[0], w5.Hg, w5.Wg), None, dev)
    hyb = time_calls(lambda i: jv.hybrid_mixers(inputs.HYBRID_SCHEDULE, lq, lk, lv, w5.Hg, w5.Wg, WIN, WIN,
                                                out=louts, ws=ws5), 3, 2, stream)
    allf = time_calls(lambda i: jv.hybrid_mixers("F" * w5.n_layers, lq, lk, lv, w5.Hg, w5.Wg, WIN, WIN,
                                                 out=louts, ws=ws5), 2, 1, stream)
    l5 = time_calls(lambda i: jv.linear_attn(lq[i % 4], lk[i % 4], lv[i % 4], w5.Hg, w5.Wg, out=lo[i % 4], ws=ws5), K, W, stream)
    w5ms = time_calls(lambda i: jv.window_attn(lq[i % 4], lk[i % 4], lv[i % 4], w5.Hg, w5.Wg, WIN, WIN, out=lo[i % 4]), K, W, stream)
    b5 = alg_bytes(*w5.shape)
    per["L@hybrid24_layer"] = {"ms": l5, "tokens_per_s": w5.tokens / (l5 * 1e-3), "GBps": b5 / l5 / 1e6, "TFLOPs": 0.0,
                               "frac_hbm": b5 / l5 / 1e6 / hbm, "frac_tensor": 0.0, "bound": "hbm"}
    f5w = alg_flops_attn(w5.B, w5.H, w5.Hg, w5.Wg, w5.D, WIN, WIN)
    per["W@hybrid24_layer"] = {"ms": w5ms, "tokens_per_s": w5.tokens / (w5ms * 1e-3), "GBps": b5 / w5ms / 1e6,
                               "TFLOPs": f5w / w5ms / 1e9, "frac_hbm": b5 / w5ms / 1e6 / hbm,
                               "frac_tensor": f5w / w5ms / 1e9 / tf, "bound": "hbm"}
    f5_flops = alg_flops_attn(w5.B, w5.H, w5.Hg, w5.Wg, w5.D, w5.Hg, w5.Wg)
    hybrid = {"schedule": inputs.HYBRID_SCHEDULE, "hybrid_ms": hyb, "all_full_ms": allf, "speedup": allf / hyb,
              "tokens_per_s_hybrid": w5.n_layers * w5.tokens / (hyb * 1e-3),
              "all_full_TFLOPs": w5.n_layers * f5_flops / allf / 1e9,
              "all_full_frac_tensor_sustained": w5.n_layers * f5_flops / allf / 1e9 / peaks["bf16_tflops_sustained"],
              "peak_note": "24 F layers back to back run under the power cap: the fraction is of the measured sustained bf16 peak",
              "note": "4 distinct layer inputs reused round-robin over the 24 layers (134 MB each: larger than L2)"}
    del q5, lo, base
    assert jv.device_status() == jv.JV_OK, "a kernel reported a timeout"

    # ---- roofline of the dominant kernel of the step: the attention kernel running F, timed inside
    # the timed region (events around the F layer of every step)
    f_ms = layer_ms[STEP_SCHEDULE.index("F")]
    f_tf = f_flops / f_ms / 1e9
    traffic, traffic_note = measured_traffic()
    roofline = {"kernel": "attn_f4_kernel as jv_full_attn (one launch per step)", "bound": "tensor", "achieved": f_tf,
                "peak": tf, "unit": "TFLOP/s", "frac": f_tf / tf, "traffic": traffic, "traffic_note": traffic_note,
                "traffic_unit": "bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum)",
                "peak_source": peaks["source"] + " bf16 burst", "ms_per_launch": f_ms,
                "flops_per_launch": f_flops, "alg_bytes_per_launch": alg_bytes(*w.shape),
                "step_layers_ms": dict(zip(["L+dwc", "W", "F"], layer_ms)),
                "linear": {"bound": "hbm", "achieved": per["L"]["GBps"], "peak": hbm, "unit": "GB/s",
                           "frac": per["L"]["GBps"] / hbm},
                "linear_dwc": {"bound": "hbm", "achieved": per["L+dwc"]["GBps"], "peak": hbm, "unit": "GB/s",
                               "frac": per["L+dwc"]["GBps"] / hbm},
                "window": {"bound": "hbm", "achieved": per["W"]["GBps"], "peak": hbm, "unit": "GB/s",
                           "frac": per["W"]["GBps"] / hbm, "tensor_frac": per["W"]["TFLOPs"] / tf}}

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample
    cpu = None
    if not args.no_cpu_baseline:
        spent, full_s, desc, cores = oracle_sample_step(w)
        cpu = {"value": step_tokens / full_s, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
               "seconds_spent": spent}

    cb = clk.summary()
    sustained["burst_ms_x_mhz"] = (ms * cb["sm_mhz"]) if cb.get("sm_mhz") else None
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "dinov3_l: 64x64 token grid (1024x1024 px, patch 16), B=8, H=16, D=64, bf16; "
                                   "one step = jv_hybrid_mixers('LWF'): L with squeeze dynamic DWC (k=3, R=128), "
                                   "W 16x16, F", "l2": "three layers' tensors (805 MB) exceed L2; "
                                   "per-mixer loops rotate over three tensor sets"},
            "clocks": clk.summary(), "sustained": sustained, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu, "per_mixer": per, "table1_variants": table1, "hybrid24": hybrid,
            "peaks": peaks}
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def run_single(args):
    """One mixer alone at a named workload shape (the command the profiler captures)."""
    from paper_2605_26636_b200 import jetvit as jv
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    w = inputs.WORKLOADS[args.workload]
    stream = torch.cuda.current_stream()
    if args.single == "F@d128":     # the workload's token count with half the heads at twice the channels
        sets = [[t.to(dev) for t in inputs.custom_qkv(w.B, max(1, w.H // 2), w.N, 128, "bf16", seed=8300 + l)] for l in range(3)]
    else:
        sets = [[t.to(dev) for t in inputs.qkv(w, layer=l)] for l in range(3)]
    outs = [torch.empty_like(s[0]) for s in sets]
    C = w.H * w.D
    dwc = None
    if args.single in ("qkv_proj", "out_proj"):
        x = inputs.normal((w.B, w.N, C), inputs.seed_for(w.cfg, 0, 5), "bf16").to(dev)
        rows = 3 * C if args.single == "qkv_proj" else C
        pw, pb = (t.to(dev) for t in inputs.proj_weights(rows, C, inputs.seed_for(w.cfg, 0, 6)))
        y = torch.empty_like(x)

        def pfn(i):
            q, k, v = sets[i % 3]
            if args.single == "qkv_proj":
                jv.qkv_proj(x, pw, pb, w.H, w.Hg, w.Wg, out=(q, k, v))
            else:
                jv.out_proj(q, pw, pb, w.Hg, w.Wg, out=y)
        ms = time_calls(pfn, args.steps, args.warmup, stream)
        assert jv.device_status() == jv.JV_OK
        print(json.dumps({"single": args.single, "workload": args.workload, "ms": ms,
                          "TFLOPs": 2.0 * w.tokens * rows * C / ms / 1e9}))
        return
    if args.single == "L+dwc":
        d = inputs.dwc_weights(C, C // 8, 3, inputs.seed_for(w.cfg, 0, 3))
        dwc = {k: (v.to(dev) if hasattr(v, "to") else v) for k, v in d.items()}
    ws = jv.alloc_workspace("L", jv.make_shape(sets[0][0], w.Hg, w.Wg), jv.make_dwc(dwc, dev), dev)

    def fn(i):
        q, k, v = sets[i % 3]
        o = outs[i % 3]
        if args.single in ("L", "L+dwc"):
            jv.linear_attn(q, k, v, w.Hg, w.Wg, dwc=dwc, out=o, ws=ws)
        elif args.single == "W":
            jv.window_attn(q, k, v, w.Hg, w.Wg, WIN, WIN, out=o)
        else:
            jv.full_attn(q, k, v, out=o)
    ms = time_calls(fn, args.steps, args.warmup, stream)
    assert jv.device_status() == jv.JV_OK
    print(json.dumps({"single": args.single, "workload": args.workload, "ms": ms,
                      "tokens_per_s": w.tokens / (ms * 1e-3)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--single", choices=["L", "L+dwc", "W", "F", "F@d128", "qkv_proj", "out_proj"], default=None,
                    help="time one mixer alone (used for profiler captures)")
    ap.add_argument("--workload", default="dinov3_l", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--record-traffic", default=None, metavar="CSV",
                    help="write the DRAM-traffic record of the dominant kernel from an ncu raw-page CSV (no GPU needed)")
    args = ap.parse_args()
    if args.record_traffic:
        record_traffic(args.record_traffic)
    elif args.single:
        run_single(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()

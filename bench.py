#!/usr/bin/env python
"""Benchmark of the fused quantized-linear hot path on B200.

A "step" is one pass of the whole hot path over one batch of synthetic input: the four quantized
linears (QKV, O, MLP-up, MLP-down) of one DiT block for one denoising step = 4 activation prologues
+ 4 low-bit GEMMs with fused epilogue (rudder_block).  Default workload: configuration 3 in NVFP4
(the largest single-GPU configuration: hidden 3072, MLP 12288, 2 x (8192 video + 64 proprio + 512
action) tokens, 10 steps of tables).  The W4A8 block (configuration 2), the W4A4-INT block
(configuration 3) and the small-M sweep (configuration 4) are measured in the same run and reported
under "also" (rank 0, N = 1).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg2_g128|cfg2_perchannel|cfg2_perchannel_static|cfg2_chained|cfg2_perchannel_static_chained|cfg3|cfg3_perchannel|cfg3_nvfp4|cfg4] [--impl reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded row sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "fused W4A8/W4A4 DiT-block linear chain throughput (2*M*K*N over QKV, O, up, down per step)"
UNIT = "TOPS"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def workload_config(name: str):
    if name == "cfg2":
        return wl.config(2)
    if name == "cfg3":
        return wl.config(3, "w4a4")
    if name == "cfg3_nvfp4":
        return wl.config(3, "nvfp4")
    if name in ("cfg2_g128", "cfg2_perchannel", "cfg2_perchannel_static"):      # configuration 2 at the other granularities
        import dataclasses
        c = wl.config(2)
        g = 128 if name == "cfg2_g128" else 0         # 0: one scale per output channel (Eq. 10 as printed)
        # "_static": one calibrated threshold per step for all rows, the activation setting of the
        # paper's sensitivity study (per-output-channel W4, static per-tensor A8)
        suffix = "_g128" if g else ("_per_channel_static" if name.endswith("_static") else "_per_channel")
        return dataclasses.replace(c, name=c.name + suffix, group=g)
    if name == "cfg2_chained":                        # configuration 2 run end to end from the QKV input (V slice, identity, GELU as glue)
        import dataclasses
        c = wl.config(2)
        return dataclasses.replace(c, name=c.name + "_chained")
    if name == "cfg2_perchannel_static_chained":      # the same chain in the paper's setting: per-channel W4, one static threshold per step;
        import dataclasses                            # the GELU then runs inside the down projection's prologue
        c = wl.config(2)
        return dataclasses.replace(c, name=c.name + "_per_channel_static_chained", group=0)
    if name == "cfg3_perchannel":                     # configuration 3 (W4A4-INT) with one scale per output channel
        import dataclasses
        c = wl.config(3, "w4a4")
        return dataclasses.replace(c, name=c.name + "_per_channel", group=0)
    raise SystemExit(f"unknown workload {name}")


def algorithmic_bytes_linear(M, K, N, G, scheme):
    """Bytes one linear must move in the two-kernel form: X, codes + r written then read, packed W +
    scales, Y, bias."""
    if scheme == "nvfp4":
        act = M * K // 2 + M * K // 16 + 4 * M
        w = N * K // 2 + N * K // 16 + 4
    else:
        # b_a bits per code: the method's 8 or 4.  (The W4A4-INT path keeps one code per BYTE in its
        # workspace, twice this: the difference shows up as traffic above the algorithmic bytes.)
        act = M * K * (8 if scheme == "w4a8" else 4) // 8 + 4 * M
        w = N * K // 2 + 2 * N * K // (G or K)       # G = 0: one scale per output channel
    return 2 * M * K + 2 * act + w + 2 * M * N + 4 * N


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 100 ms in the background."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()

    def summary(self, t0, t1):
        sm, smax, reasons = [], 0.0, set()
        for t, line in self.samples:
            if t < t0 or t > t1:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax = max(smax, float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": smax, "reasons": sorted(reasons), "samples": len(sm)}


def build_block(rd, cfg, torch, dev):
    """Pack the four weights and put the replay inputs of one block on the device."""
    lins = cfg.draw()
    scheme = rd.SCHEMES[cfg.scheme]
    ws, tabs, biases, xs, ys, keep = [], [], [], [], [], []
    for l in lins:
        W = torch.from_numpy(l.W).to(dev)
        d = torch.from_numpy(l.d).to(dev)
        ws.append(rd.rudder_pack_weights(W, d, scheme, cfg.group or l.K))     # group 0: one scale per output channel (G = K)
        del W, d
        gamma = torch.from_numpy(l.gamma).to(dev)
        if cfg.name.endswith("_static") or cfg.name.endswith("_static_chained"):
            # input recipe, step 8: clip[t] = 99.9th percentile of |(x dinv) gamma[t, s(i)]| over all rows
            x = torch.from_numpy(l.X_bf16.view(np.int16)).to(dev).view(torch.bfloat16).float()
            x *= rd.rudder_weight_export(ws[-1])["dinv"][None, :]
            row_stream = torch.from_numpy(np.repeat(l.seg_stream, np.diff(l.seg_offsets)).astype(np.int64)).to(dev)
            k = max(1, int(round(0.999 * x.numel())))
            clip = torch.stack([torch.kthvalue((x * gamma[t][row_stream][:, None]).abs().flatten(), k).values
                                for t in range(gamma.shape[0])]).float().contiguous()
            del x
            tabs.append(rd.ScaleTable(gamma, clip, rd.RANGE_STATIC))
        else:
            tabs.append(rd.ScaleTable(gamma, None, rd.RANGE_PER_TOKEN))
        biases.append(torch.from_numpy(l.bias).to(dev))
        xs.append(torch.from_numpy(l.X_bf16.view(np.int16)).to(dev).view(torch.bfloat16))
        ys.append(torch.empty((l.M, l.N), dtype=torch.bfloat16, device=dev))
    seg = rd.Segments(lins[0].seg_offsets, lins[0].seg_stream)
    if cfg.name.endswith("_chained"):
        xs = [xs[0], None, None, None]               # layers 1..3 read the previous output through the BF16 glue
    return lins, ws, tabs, biases, xs, ys, seg


# DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum from one
# ncu capture of that launch; summaries under profiles/).  Keyed by workload; None = not captured.
NCU_TRAFFIC_BYTES = {
    # sum over the kernel's 4 launches of one step (profiles/gemm_nvfp4_and_actq_cfg3_metrics.md,
    # profiles/gemm_i8_w4_and_actq_cfg2_metrics.md, profiles/gemm_i8_w4_f8_and_actq_cfg3_w4a4_metrics.md)
    "cfg3_nvfp4_block_h3072_f12288_m17536": 1287.4e6,
    "cfg2_w4a8_block_h2048_f8192_m4416": 119.2e6,
    "cfg3_w4a4_block_h3072_f12288_m17536": 1791.5e6,
}


NOMINAL_TOPS = {"w4a8": 4500.0, "w4a4": 4500.0, "nvfp4": 9000.0}     # datasheet dense INT8 / FP4 rates of a B200


def bf16_block_ms(torch, cfg, xs_shapes, dev, reps=10):
    """cuBLAS BF16 GEMMs (torch.matmul) on the same four shapes, back to back: the speed-up reference."""
    M = cfg.M
    xb = [torch.randn((M, K), dtype=torch.bfloat16, device=dev) for _, K, N in cfg.linears]
    wbf = [torch.randn((N, K), dtype=torch.bfloat16, device=dev) for _, K, N in cfg.linears]
    for _ in range(3):
        for x, w_ in zip(xb, wbf):
            torch.matmul(x, w_.t())
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        for x, w_ in zip(xb, wbf):
            torch.matmul(x, w_.t())
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def measure_block(rd, torch, dev, cfg, steps, warmup, world=1, rank=0, dist=None, sampler=None, sustain_s=2.0):
    """Two timed legs of one workload.  (1) `steps` block passes after `warmup`, CUDA events, max over ranks:
    the line's ms_per_step.  (2) a sustained leg: the same pass repeated for at least `sustain_s` seconds in
    chunks timed by CUDA events, with one per-kernel profile pass (an event between launches) after every
    chunk, so that the per-kernel times are taken in the same thermal and clock state as the step time they
    are reported beside.  Clocks are sampled for each leg."""
    from paper_2609_39056_b200.dist_util import max_over_ranks
    M, T = cfg.M, cfg.T
    lins, ws, tabs, biases, xs, ys, seg = build_block(rd, cfg, torch, dev)
    bargs = rd.BlockArgs(ws, tabs, biases, xs, ys)
    workspace = torch.empty(rd.rudder_block_workspace_bytes(bargs, M) + 256, dtype=torch.uint8, device=dev)
    ops = cfg.ops()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        rd.rudder_block(bargs, M, seg, i % T, workspace)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record()
    for i in range(steps):
        rd.rudder_block(bargs, M, seg, i % T, workspace)
    ev1.record()
    barrier()
    t_wall1 = time.time()
    ms_per_step = max_over_ranks(ev0.elapsed_time(ev1), dev) / steps
    clocks = sampler.summary(t_wall0, t_wall1) if sampler is not None else None

    # ---- sustained leg
    chunk = max(10, min(100, int(0.05 / max(ms_per_step * 1e-3, 1e-6))))       # about 50 ms of steps per chunk
    prof = np.zeros(8)
    n_prof, n_steps, ms_sum = 0, 0, 0.0
    t_s0 = time.time()
    while time.time() - t_s0 < sustain_s or n_prof < 3:
        ev0.record()
        for i in range(chunk):
            rd.rudder_block(bargs, M, seg, i % T, workspace)
        ev1.record()
        ev1.synchronize()
        ms_sum += ev0.elapsed_time(ev1)
        n_steps += chunk
        prof += np.array(rd.rudder_block_profile(bargs, M, seg, n_prof % T, workspace))
        n_prof += 1
    t_s1 = time.time()
    prof /= n_prof
    sus_ms = max_over_ranks(ms_sum / n_steps, dev)
    sus_clocks = sampler.summary(t_s0, t_s1) if sampler is not None else None
    if clocks is None or clocks.get("samples", 0) < 3:
        # the first leg is shorter than the sampling period: its clock record is the sustained leg's
        clocks = dict(sus_clocks) if sus_clocks else None
        if clocks is not None:
            clocks["note"] = "timed region shorter than the sampling period: sampled over the sustained leg that follows it"
    status, where = rd.rudder_device_status()
    if status != 0:
        raise SystemExit(f"device status {status} (wait {where}): the run is invalid")
    sustained = {"ms_per_step": sus_ms, "tops": ops / (sus_ms * 1e-3) / 1e12, "steps": n_steps, "seconds": t_s1 - t_s0,
                 "clocks": sus_clocks, "profile_passes": n_prof}
    return dict(cfg=cfg, lins=lins, ws=ws, tabs=tabs, biases=biases, xs=xs, ys=ys, seg=seg, workspace=workspace,
                ops=ops, ms_per_step=ms_per_step, clocks=clocks, prof=prof, sustained=sustained)


def roofline_of(cfg, m, pk):
    """Roofline object of the dominant kernel (the GEMM: 4 launches per step).  The per-kernel times come from
    the profile passes of the sustained leg (an event between launches, which also keeps consecutive kernels
    from overlapping): they are scaled so that prologues + GEMMs add up to that leg's step time, and the
    fractions divide by the SUSTAINED measured peak (the kernel runs inside a seconds-long loop) and, beside
    it, by the datasheet dense rate."""
    M = cfg.M
    sus = m["sustained"]
    raw_gemm, raw_actq, raw_sum = float(m["prof"][1::2].sum()), float(m["prof"][0::2].sum()), float(m["prof"].sum())
    scale = sus["ms_per_step"] / raw_sum
    gemm_ms, actq_ms = raw_gemm * scale, raw_actq * scale
    ratio = 4.0 if cfg.scheme == "nvfp4" else 2.0          # FP4 / INT8 dense rate relative to bf16
    tensor_peak = ratio * pk["bf16_sustained"]
    nominal = NOMINAL_TOPS[cfg.scheme]
    achieved = m["ops"] / (gemm_ms * 1e-3) / 1e12
    if cfg.scheme == "nvfp4":
        pro_bytes = sum(2 * M * K + M * K // 2 + M * K // 16 + 4 * M for _, K, N in cfg.linears)
    else:
        pro_bytes = sum(2 * M * K + M * K * (8 if cfg.scheme == "w4a8" else 4) // 8 + 4 * M for _, K, N in cfg.linears)
    traffic = NCU_TRAFFIC_BYTES.get(cfg.name)
    sm_mhz = (sus["clocks"] or {}).get("sm_mhz")
    return {"kernel": "gemm_nvfp4_pair_kernel" if cfg.scheme == "nvfp4" else "gemm_i8_w4_kernel", "launches_per_step": 4,
            "bound": "tensor", "achieved": achieved, "peak": tensor_peak,
            "unit": "TFLOP/s" if cfg.scheme == "nvfp4" else "TOPS", "frac": achieved / tensor_peak,
            "peak_source": f"{pk['source']} bf16 SUSTAINED {pk['bf16_sustained']} x {ratio:g} (nominal ratio), of measured; the kernel is timed inside the sustained leg",
            "frac_of_nominal_dense": achieved / nominal, "nominal_dense_peak": nominal,
            "frac_of_burst_measured": achieved / (ratio * pk["bf16_burst"]),
            "sm_mhz_median": sm_mhz, "leg": "sustained",
            "traffic": traffic, "gemm_ms": gemm_ms, "prologue_ms": actq_ms, "step_ms_of_leg": sus["ms_per_step"],
            "profile_raw_ms": {"gemm": raw_gemm, "prologue": raw_actq,
                               "note": "as measured with an event between launches; scaled by step_ms_of_leg / their sum"},
            "prologue": {"bound": "hbm", "achieved": pro_bytes / (actq_ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                         "frac": pro_bytes / (actq_ms * 1e-3) / 1e9 / pk["hbm_gbs"]},
            "per_kernel_ms": [float(v) * scale for v in m["prof"]]}


def _graph_us(torch, stream, calls):
    """Median device time (us) per call of a CUDA graph holding `calls` (a list of closures), 5 warm-up + 20 timed replays."""
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for c in calls:
                c()
        for _ in range(5):
            graph.replay()
        stream.synchronize()
        times = []
        for _ in range(20):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            e1.synchronize()
            times.append(e0.elapsed_time(e1) / len(calls))
    return float(np.median(times)) * 1e3


def small_m_sweep(rd, torch, dev, pk, schemes=("w4a8", "w4a4"), sizes=(2048, 4096), rows=(16, 64, 128, 256), cold=True):
    """Configuration 4: action + proprio-only passes.  (i) One packed weight reused across 20 steps, captured
    in one CUDA graph (weights stay L2-resident: `algorithmic` GB/s counts every byte the call must move).
    (ii) `cold`: the same call over a rotation of distinct packed weights whose total size is several
    times the L2 (at least 64 of them), one graph of one linear per weight: every weight comes from HBM,
    as in a model whose layers do not fit the cache."""
    out = []
    L2_BYTES = 126e6
    for scheme in schemes:
        for KN in sizes:
            for M in rows:
                cfg = wl.config(4, scheme, M=M, KN=KN)
                l = cfg.draw()[0]
                W = torch.from_numpy(l.W).to(dev)
                d = torch.from_numpy(l.d).to(dev)
                w = rd.rudder_pack_weights(W, d, rd.SCHEMES[scheme], cfg.group)
                tab = rd.ScaleTable(torch.from_numpy(l.gamma).to(dev), None, rd.RANGE_PER_TOKEN)
                seg = rd.Segments(l.seg_offsets, l.seg_stream)
                X = torch.from_numpy(l.X_bf16.view(np.int16)).to(dev).view(torch.bfloat16)
                bias = torch.from_numpy(l.bias).to(dev)
                Y = torch.empty((M, KN), dtype=torch.bfloat16, device=dev)
                ws = torch.empty(rd.rudder_linear_workspace_bytes(w, M) + 256, dtype=torch.uint8, device=dev)
                stream = torch.cuda.Stream()
                with torch.cuda.stream(stream):
                    for t in range(3):
                        rd.rudder_linear(w, X, seg, t, tab, bias, Y=Y, workspace=ws)
                    stream.synchronize()
                us = _graph_us(torch, stream, [
                    (lambda t=t: rd.rudder_linear(w, X, seg, t, tab, bias, Y=Y, workspace=ws)) for t in range(cfg.T)])
                nbytes = algorithmic_bytes_linear(M, KN, KN, cfg.group, scheme)
                # cuBLAS BF16 on the same shape under the same protocol (one weight, 20 calls in one graph)
                Wb = torch.randn((KN, KN), dtype=torch.bfloat16, device=dev)
                Yb = torch.empty((M, KN), dtype=torch.bfloat16, device=dev)
                with torch.cuda.stream(stream):
                    for _ in range(3):
                        torch.matmul(X, Wb.t(), out=Yb)
                    stream.synchronize()
                us_bf16 = _graph_us(torch, stream, [(lambda: torch.matmul(X, Wb.t(), out=Yb)) for _ in range(cfg.T)])
                del Wb, Yb
                row = {"scheme": scheme, "M": M, "K": KN, "N": KN, "us_per_linear": us, "us_bf16_cublas": us_bf16,
                       "x_bf16": us_bf16 / us,
                       "algorithmic_gbs": nbytes / (us * 1e-6) / 1e9, "hbm_frac": nbytes / (us * 1e-6) / 1e9 / pk["hbm_gbs"],
                       "tops": 2.0 * M * KN * KN / (us * 1e-6) / 1e12}
                if cold:
                    w_bytes = KN * KN // 2 + (KN // cfg.group) * KN * 6        # codes + fp32 and fp16 scale copies
                    n_w = max(64, int(np.ceil(3 * L2_BYTES / w_bytes)))
                    rotation = [w] + [rd.rudder_pack_weights(W, d, rd.SCHEMES[scheme], cfg.group) for _ in range(n_w - 1)]
                    us_c = _graph_us(torch, stream, [
                        (lambda i=i: rd.rudder_linear(rotation[i], X, seg, i % cfg.T, tab, bias, Y=Y, workspace=ws))
                        for i in range(n_w)])
                    row.update({"cold_weights": n_w, "us_per_linear_cold": us_c,
                                "algorithmic_gbs_cold": nbytes / (us_c * 1e-6) / 1e9,
                                "hbm_frac_cold": nbytes / (us_c * 1e-6) / 1e9 / pk["hbm_gbs"]})
                    del rotation
                out.append(row)
                del w
    return out


def crossattn_kv(rd, torch, dev, pk, schemes=("w4a8", "w4a4", "nvfp4")):
    """The cross-attention key / value projections (one global-text region each): both linears of one step in a CUDA
    graph over the 10 steps of tables, microseconds per pair, cuBLAS BF16 on the same shapes beside it."""
    out = []
    for scheme in schemes:
        cfg = wl.config(5, scheme)
        lins = cfg.draw()
        items = []
        for l in lins:
            W = torch.from_numpy(l.W).to(dev)
            d = torch.from_numpy(l.d).to(dev)
            w = rd.rudder_pack_weights(W, d, rd.SCHEMES[scheme], cfg.group)
            items.append(dict(w=w, tab=rd.ScaleTable(torch.from_numpy(l.gamma).to(dev), None, rd.RANGE_PER_TOKEN),
                              X=torch.from_numpy(l.X_bf16.view(np.int16)).to(dev).view(torch.bfloat16), bias=torch.from_numpy(l.bias).to(dev),
                              Y=torch.empty((l.M, l.N), dtype=torch.bfloat16, device=dev),
                              ws=torch.empty(rd.rudder_linear_workspace_bytes(w, l.M) + 256, dtype=torch.uint8, device=dev),
                              Wb=torch.randn((l.N, l.K), dtype=torch.bfloat16, device=dev)))
        seg = rd.Segments(lins[0].seg_offsets, lins[0].seg_stream)
        stream = torch.cuda.Stream()

        def pair(t):
            for it in items:
                rd.rudder_linear(it["w"], it["X"], seg, t, it["tab"], it["bias"], Y=it["Y"], workspace=it["ws"])

        def pair_bf16():
            for it in items:
                torch.matmul(it["X"], it["Wb"].t(), out=it["Y"])

        with torch.cuda.stream(stream):
            for t in range(3):
                pair(t)
                pair_bf16()
            stream.synchronize()
        us = _graph_us(torch, stream, [(lambda t=t: pair(t)) for t in range(cfg.T)])
        us_b = _graph_us(torch, stream, [pair_bf16 for _ in range(cfg.T)])
        ops = cfg.ops()
        out.append({"workload": cfg.name, "scheme": scheme, "us_per_pair": us, "tops": ops / (us * 1e-6) / 1e12,
                    "us_bf16_cublas": us_b, "x_bf16": us_b / us})
    return out


def calibrator_timing(rd, torch, dev):
    """Toy calibrator (Eq. 9) on the QKV layer of configuration 2, one layer-step: wall time of the whole
    search (every candidate is one static-mode rudder_linear plus the error reduction)."""
    from paper_2609_39056_b200 import calibrate as gc
    cfg = wl.config(2)
    l = cfg.draw()[0]
    W = torch.from_numpy(l.W).to(dev)
    d = torch.from_numpy(l.d).to(dev)
    w = rd.rudder_pack_weights(W, d, rd.SCHEMES[cfg.scheme], l.K)           # one scale per output channel
    X = torch.from_numpy(l.X_bf16.view(np.int16)).to(dev).view(torch.bfloat16)
    seg = rd.Segments(l.seg_offsets, l.seg_stream)
    v = (X.float() * rd.rudder_weight_export(w)["dinv"][None, :]).abs().flatten()
    cs = [float(torch.kthvalue(v, max(1, int(round(q * v.numel())))).values) for q in (0.99, 0.999, 0.9999, 1.0)]
    steps = [2 ** -0.5, 2 ** -0.25, 2 ** 0.25, 2 ** 0.5]
    gc.calibrate_step(w, X, seg, 3, cs[:1], steps[:1], sweeps=1)            # warm-up
    torch.cuda.synchronize()
    t0 = time.time()
    r = gc.calibrate_step(w, X, seg, 3, cs, steps)
    torch.cuda.synchronize()
    dt = time.time() - t0
    return {"layer": "cfg2 qkv 4416x2048x6144, per-channel W4A8, static range", "ms": dt * 1e3, "evaluations": r["evaluations"],
            "gamma": [float(g) for g in r["gamma"]], "clip": r["clip"], "objective": r["objective"]}


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    import paper_2609_39056_b200 as rd
    from paper_2609_39056_b200.dist_util import max_over_ranks, whole_job_value
    rd.lib()
    pk = peaks()

    if args.workload == "cfg4":
        # Configuration 4 alone (the small-M sweep that the default run reports under "also"): the command
        # the ncu summary of the small-M kernels is taken from.  Rank 0 only; the value is the sweep's
        # mean throughput.
        if rank == 0:
            sweep = small_m_sweep(rd, torch, dev, pk, schemes=tuple(args.cfg4_schemes.split(",")), sizes=tuple(int(x) for x in args.cfg4_sizes.split(",")),
                                  rows=tuple(int(x) for x in args.cfg4_rows.split(",")), cold=not args.no_cold)
            mean_us = float(np.mean([r["us_per_linear"] for r in sweep]))
            print(json.dumps({"metric": "small-M W4A8 linear (configuration 4), mean over M in {16,64,128,256}, K=N in {2048,4096}",
                              "value": float(np.mean([r["tops"] for r in sweep])), "unit": "TOPS", "n_gpus": 1,
                              "steps": 20, "warmup": 5, "ms_per_step": mean_us * 1e-3, "higher_is_better": True,
                              "scaling": "weak", "vs_baseline": None, "dtype": "int8 x int4 -> int32", "data": "synthetic",
                              "config": {"workload": "cfg4_small_m_sweep"}, "sweep": sweep}))
        if world > 1:
            dist.destroy_process_group()
        return
    cfg = workload_config(args.workload)
    M, T = cfg.M, cfg.T
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler is not None:
        sampler.start()
    m = measure_block(rd, torch, dev, cfg, args.steps, args.warmup, world, rank, dist, sampler, sustain_s=args.sustain_seconds)
    ops, ms_per_step = m["ops"], m["ms_per_step"]
    clocks_main = m["clocks"]
    sustained_main = m["sustained"]
    value = whole_job_value(ops, world, ms_per_step) / 1e12
    roofline = roofline_of(cfg, m, pk)
    alg_bytes = [algorithmic_bytes_linear(M, K, N, cfg.group, cfg.scheme) for _, K, N in cfg.linears]
    ws, tabs, biases, xs, ys, seg, workspace, lins = (m[k] for k in ("ws", "tabs", "biases", "xs", "ys", "seg", "workspace", "lins"))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- end to end through the C ABI with HOST buffers (pinned): H2D of the 4 inputs, block, D2H of the 4 outputs
    if cfg.name.endswith("_chained"):                # the host-buffer entry point replays four inputs: time the replay form of the same block
        xs = [torch.from_numpy(l.X_bf16.view(np.int16)).to(dev).view(torch.bfloat16) for l in lins]
    hx = [x.cpu().pin_memory() for x in xs]
    hy = [torch.empty(y.shape, dtype=y.dtype).pin_memory() for y in ys]
    hargs = rd.BlockArgs(ws, tabs, biases, hx, hy)
    staging = torch.empty(rd.rudder_block_host_staging_bytes(hargs, M) + 256, dtype=torch.uint8, device=dev)
    e2e_steps = max(3, min(args.steps, 10))
    for i in range(2):
        rd.rudder_block_host(hargs, M, seg, i % T, staging, workspace)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(e2e_steps):
        rd.rudder_block_host(hargs, M, seg, i % T, staging, workspace)
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1) / e2e_steps, dev)
    h2d = sum(int(x.numel()) * 2 for x in hx)
    d2h = sum(int(y.numel()) * 2 for y in hy)
    e2e = {"value": whole_job_value(ops, world, e2e_ms) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    del staging, hx, hy, hargs

    # ---- cuBLAS BF16 on the same shapes (speed-up reference only)
    bf16_ms = None
    if rank == 0 and not args.no_bf16:
        bf16_ms = bf16_block_ms(torch, cfg, None, dev)

    # ---- the oracle on this machine's host cores, on a bounded row sample (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(cfg, lins, target_s=args.cpu_seconds)

    # ---- the other workloads of the metric, briefly (rank 0, N = 1 only)
    also = None
    if rank == 0 and world == 1 and not args.no_also:
        del m, ws, tabs, biases, xs, ys, workspace, lins
        torch.cuda.empty_cache()
        also = {}
        for name in ("cfg2", "cfg2_g128", "cfg2_perchannel", "cfg2_perchannel_static", "cfg2_chained", "cfg2_perchannel_static_chained", "cfg3", "cfg3_perchannel",
                     "cfg3_nvfp4"):
            if name == args.workload:
                continue
            c2 = workload_config(name)
            m2 = measure_block(rd, torch, dev, c2, max(10, min(args.steps, 50)), 5, sampler=sampler, sustain_s=args.sustain_seconds)
            r2 = roofline_of(c2, m2, pk)
            b2 = bf16_block_ms(torch, c2, None, dev) if not args.no_bf16 else None
            also[c2.name] = {"ms_per_step": m2["ms_per_step"], "us_per_block_step": m2["ms_per_step"] * 1e3,
                             "tops": c2.ops() / (m2["ms_per_step"] * 1e-3) / 1e12, "sustained": m2["sustained"],
                             "gemm_frac_of_tensor_peak": r2["frac"], "gemm_frac_of_nominal_dense": r2["frac_of_nominal_dense"],
                             "gemm_achieved": r2["achieved"], "gemm_peak": r2["peak"], "prologue_hbm_frac": r2["prologue"]["frac"],
                             "per_kernel_ms": r2["per_kernel_ms"], "bf16_cublas_ms_per_step": b2,
                             "x_bf16": (b2 / m2["sustained"]["ms_per_step"]) if b2 else None}
            del m2
            torch.cuda.empty_cache()
        also["cfg4_small_m_sweep"] = small_m_sweep(rd, torch, dev, pk)
        also["cfg5_crossattn_kv"] = crossattn_kv(rd, torch, dev, pk)
        also["toy_calibrator"] = calibrator_timing(rd, torch, dev)
    if sampler is not None:
        sampler.stop()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "us_per_block_step": ms_per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": {"w4a8": "int8 x int4 -> int32", "w4a4": "int4 x int4 -> int32",
                                                              "nvfp4": "e2m1 x e2m1 (ue4m3 block scales) -> fp32"}[cfg.scheme],
            "data": "synthetic", "gpu_launches": 8 * args.steps,
            "config": {"workload": cfg.name, "scheme": cfg.scheme, "group": 16 if cfg.scheme == "nvfp4" else cfg.group, "M": M,
                       "linears": {n: [K, N] for n, K, N in cfg.linears}, "range_mode": "static" if "_static" in cfg.name else "per_token",
                       "steps_of_tables": T, "tops_per_step": ops / 1e12,
                       "l2": f"working set per step {sum(alg_bytes) / 1e6:.0f} MB (inputs {sum(2 * M * K for _, K, _ in cfg.linears) / 1e6:.0f} MB) exceeds the 126 MB L2; no explicit flush",
                       "parallelism": f"replicas x{world} (rows independent, no collective)"},
            "clocks": m_clocks(locals()), "e2e": e2e, "roofline": roofline, "cpu_baseline": cpu,
            "bf16_cublas_ms_per_step": bf16_ms,
            "speedup_vs_bf16_cublas": (bf16_ms / ms_per_step) if bf16_ms else None,
            "algorithmic_mb_per_step": sum(alg_bytes) / 1e6,
            "paper_context": "paper reports up to 2.23x denoising speed-up over BF16 (W4A4) and 1.35x end to end (W4A8), both on an RTX 4090: context, not the target",
            "also": also,
        }
        line["sustained"] = sustained_main
        line["speedup_vs_bf16_cublas_sustained"] = (bf16_ms / sustained_main["ms_per_step"]) if bf16_ms else None
        line["summary"] = make_summary(cfg, sustained_main, roofline, bf16_ms, also)      # last key: short enough to survive a truncated log
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def make_summary(cfg, sustained, roofline, bf16_ms, also):
    """Compact digest: per block workload [sustained ms per step, TOPS, GEMM fraction of the sustained measured
    peak, of the nominal dense peak, speed-up over cuBLAS BF16]; per small-M point [us per linear, fraction of
    the measured HBM bandwidth, speed-up over cuBLAS BF16]."""
    r3 = lambda v: None if v is None else float(f"{v:.3g}")
    out = {"keys": "block: [ms_sustained, TOPS, gemm_frac_sustained_peak, gemm_frac_nominal, x_bf16]; cfg4: {scheme_K: {M: [us, hbm_frac, x_bf16]}}; cfg5: {scheme: [us_per_kv_pair, TOPS, x_bf16]}"}
    tag = lambda name: name.split("_block")[0] + name.split("m4416")[-1].split("m17536")[-1]
    out[tag(cfg.name)] = [r3(sustained["ms_per_step"]), r3(sustained["tops"]), r3(roofline["frac"]), r3(roofline["frac_of_nominal_dense"]),
                          r3(bf16_ms / sustained["ms_per_step"]) if bf16_ms else None]
    for name, v in (also or {}).items():
        if isinstance(v, dict) and "sustained" in v:
            out[tag(name)] = [r3(v["sustained"]["ms_per_step"]), r3(v["sustained"]["tops"]), r3(v["gemm_frac_of_tensor_peak"]),
                              r3(v["gemm_frac_of_nominal_dense"]), r3(v["x_bf16"])]
    sweep = (also or {}).get("cfg4_small_m_sweep")
    if sweep:
        c4 = {}
        for r in sweep:
            c4.setdefault(f"{r['scheme']}_{r['K']}", {})[str(r["M"])] = [r3(r["us_per_linear"]), r3(r["hbm_frac"]), r3(r.get("x_bf16"))]
        out["cfg4"] = c4
    ca = (also or {}).get("cfg5_crossattn_kv")
    if ca:
        out["cfg5_crossattn_kv"] = {r["scheme"]: [r3(r["us_per_pair"]), r3(r["tops"]), r3(r["x_bf16"])] for r in ca}
    return out


def m_clocks(loc):
    return loc.get("clocks_main")


def cpu_baseline(cfg, lins, target_s=15.0, impl_reference=False):
    """Time the oracle, as it stands, on a bounded sample of rows of the same workload."""
    import oracle
    cores = oracle.num_threads()
    packs = []
    for l in lins:
        packs.append(oracle.pack_nvfp4(l.W, l.d) if cfg.scheme == "nvfp4" else oracle.pack_int4(l.W, l.d, cfg.group or l.K))
    M = cfg.M
    static = "_static" in cfg.name
    clips = []
    for l, pw in zip(lins, packs):
        if not static:
            clips.append(None)
            continue
        # the workload's threshold (99.9th percentile of |(x dinv) gamma|), here from every 16th row: the
        # oracle's time does not depend on its value
        X = wl.bf16_bits_to_f32(l.X_bf16[::16])
        st = np.repeat(l.seg_stream, np.diff(l.seg_offsets))[::16]
        clips.append(np.array([np.percentile(np.abs((X * pw["dinv"][None, :]) * l.gamma[t, st][:, None]), 99.9)
                               for t in range(l.gamma.shape[0])], np.float32))

    def run(rows):
        t0 = time.time()
        for l, pw, clip in zip(lins, packs, clips):
            oracle.rudder_linear(l.X_bf16, pw, l.gamma, clip, 0, oracle.RANGE_STATIC if static else oracle.RANGE_PER_TOKEN,
                                 l.seg_offsets, l.seg_stream, cfg.scheme, l.bias, rows=rows)
        return time.time() - t0

    rng = np.random.default_rng(1234)
    n0 = min(M, 4 * cores)
    t_probe = run(np.sort(rng.choice(M, n0, replace=False)).astype(np.int32))
    n = int(min(M, max(n0, n0 * target_s / max(t_probe, 1e-3))))
    n = max(cores, n // cores * cores)
    rows = np.sort(rng.choice(M, n, replace=False)).astype(np.int32)
    t = run(rows)
    ops_sample = sum(2.0 * n * K * N for _, K, N in cfg.linears)
    return {"value": ops_sample / t / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} of {M} rows (seeded), all four linears, step 0, {t:.1f} s wall", "seconds": t}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = workload_config(args.workload)
    lins = cfg.draw()
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    res = None
    times = []
    for i in range(args.warmup + args.steps):
        res = cpu_baseline(cfg, lins, target_s=per_step)
        if i >= args.warmup:
            times.append(res["value"])
    value = float(np.mean(times))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["seconds"] * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "oracle (fp32 / int32 / fp64 on CPU)", "data": "synthetic",
            "config": {"workload": cfg.name, "scheme": cfg.scheme, "group": 16 if cfg.scheme == "nvfp4" else cfg.group, "M": cfg.M,
                       "linears": {n: [K, N] for n, K, N in cfg.linears}},
            "cpu_baseline": {"kind": "oracle", "cores": res["cores"], "sample": res["sample"], "value": value, "unit": UNIT},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_nvfp4")
    ap.add_argument("--no-also", action="store_true", help="skip the other workloads reported under \"also\"")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline leg")
    ap.add_argument("--no-bf16", action="store_true", help="skip the cuBLAS BF16 comparison")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--cfg4-schemes", default="w4a8", help="--workload cfg4: schemes of the sweep")
    ap.add_argument("--cfg4-sizes", default="2048,4096", help="--workload cfg4: K = N values")
    ap.add_argument("--cfg4-rows", default="16,64,128,256", help="--workload cfg4: M values")
    ap.add_argument("--no-cold", action="store_true", help="--workload cfg4: skip the rotation over distinct weights")
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="length of the sustained leg of every block workload")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

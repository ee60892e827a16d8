#!/usr/bin/env python
"""Benchmark of the CRISP hybrid-sparse hot path on B200.

One *step* = the whole path on one layer: crisp_build_mask (saliency -> hybrid mask),
crisp_encode (weight + mask -> compressed format + execution image) and crisp_spmm
(Y = W_hybrid X), all through the C ABI.  The headline metric is useful TFLOP/s of the
step, 2 * nnz * ncols / step time; the SpMM kernel alone, its roofline fraction and its
speedup over a dense bf16 cuBLAS GEMM of the same shape are reported beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints exactly one JSON line on rank 0.
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
sys.path.insert(0, ROOT)

from paper_2311_14272_b200 import workloads as wl  # noqa: E402

METRIC = "hybrid_sparse_spmm_useful_tflops"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_FLUSH_BYTES = 256 << 20


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def pick_layer(name: str) -> wl.Layer:
    if name == "config2":
        return wl.config2()[0]
    if name == "config1":
        return wl.config1()[0]
    if name.startswith("sweep_"):
        nm, keep = name[len("sweep_"):].split("_keep")
        n, m = nm.split(":")
        return wl.sweep_cell(int(n), int(m), float(keep))
    for l in wl.config3() + wl.config4():
        if l.name == name:
            return l
    raise SystemExit(f"unknown workload {name}")


# --------------------------------------------------------------------- clock sampling

class ClockSampler:
    """Samples SM clock and throttle reasons while the timed region runs.

    NVML is read in-process (a sample costs microseconds, so even a timed region of a few milliseconds is
    covered): by a thread every 0.5 ms and by `sample()` calls of the main thread while it waits for the queued steps
    to finish (the timed steps are queued behind untimed work, so no launch waits for a host call).  Where NVML cannot
    be loaded, `nvidia-smi -lms` is read instead.  Reading only: no setting of the GPU is touched.
    """
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.proc = None
        self.lines = []
        self.nv = None
        self.handle = None
        self.sm, self.smax, self.reasons = [], [], set()
        self._stop = threading.Event()
        self._lock = threading.Lock()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def sample(self):
        nv = self.nv
        if nv is None:
            return
        try:
            mhz = float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
            bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
        except Exception:
            return
        with self._lock:
            self.sm.append(mhz)
            self.smax.append(self.max_mhz)
            for nm, bit in (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40),
                            ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4)):
                if bits & bit:
                    self.reasons.add(nm)

    def _poll(self):
        while not self._stop.is_set():
            self.sample()
            time.sleep(0.0005)

    def start(self):
        if self.nv is not None:
            self.t = threading.Thread(target=self._poll, daemon=True)
            self.t.start()
            return
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.nv is not None:
            self._stop.set()
            self.t.join(timeout=1)
            return {"sm_mhz": float(np.median(self.sm)) if self.sm else None,
                    "sm_max_mhz": float(max(self.smax)) if self.smax else None,
                    "samples": len(self.sm), "reasons": sorted(self.reasons), "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi"}


# ------------------------------------------------------------------------ CPU oracle

def oracle_step(layer, w, s, x_sample):
    """One pass of the oracle as it stands on a bounded column sample; returns (seconds, nnz)."""
    import oracle
    t0 = time.perf_counter()
    mk = oracle.build_mask(s, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio)
    vals, idx = oracle.encode(w, mk)
    wd, _ = oracle.decode(mk.blk_col, vals, idx, layer.rows, layer.k, layer.n, layer.m,
                          layer.block_rows, layer.block_k, mk.kkeep)
    oracle.spmm_fp64(wd, x_sample)
    return time.perf_counter() - t0, int(vals.size)


def oracle_sample_cols(layer, w, s, x, target_s=12.0):
    """Choose how many columns of X the oracle multiplies so that one pass takes ~target_s."""
    import oracle
    mk = oracle.build_mask(s, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio)
    vals, idx = oracle.encode(w, mk)
    wd, _ = oracle.decode(mk.blk_col, vals, idx, layer.rows, layer.k, layer.n, layer.m,
                          layer.block_rows, layer.block_k, mk.kkeep)
    pc = min(256, x.shape[1])
    probe = np.ascontiguousarray(x[:, :pc])
    t0 = time.perf_counter()
    oracle.spmm_fp64(wd, probe)
    per_col = (time.perf_counter() - t0) / pc
    return int(max(4, min(x.shape[1], 1024, target_s / max(per_col, 1e-9))))


def run_reference(args, layer, rank):
    """--impl reference: the CPU oracle, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import oracle
    w, s, x = wl.make_layer_inputs(layer)
    cols = oracle_sample_cols(layer, w, s, x, target_s=max(2.0, 60.0 / max(1, args.steps + args.warmup)))
    xs = np.ascontiguousarray(x[:, :cols])
    for _ in range(args.warmup):
        oracle_step(layer, w, s, xs)
    tot, nnz = 0.0, 0
    for _ in range(args.steps):
        dt, nnz = oracle_step(layer, w, s, xs)
        tot += dt
    ms = tot / args.steps * 1e3
    value = 2.0 * nnz * cols / (ms * 1e-3) / 1e12
    sample = f"mask+encode+decode of the full layer, fp64 product on the first {cols} of {layer.ncols} columns"
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": args.workload, "rows": layer.rows, "k": layer.k, "ncols": layer.ncols,
                      "sampled_ncols": cols},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


# ---------------------------------------------------------------------------- GPU arm

def roofline_terms(model, peaks, spmm_ms, ncols):
    """Slot-aware tensor time and algorithmic-byte HBM time of one crisp_spmm call."""
    useful = 2.0 * model["nnz"] * ncols
    slot_flops = 2.0 * model["slot_macs"]
    hbm_bytes = model["vals_bytes"] + model["idx_bytes"] + model["blk_col_bytes"] + model["x_bytes"] + model["y_bytes"]
    t_tensor = slot_flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = hbm_bytes / (peaks["hbm_gbs"] * 1e9)
    return {"useful_flops": useful, "slot_flops": slot_flops, "hbm_bytes": hbm_bytes, "t_tensor": t_tensor,
            "t_hbm": t_hbm, "frac": max(t_tensor, t_hbm) / (spmm_ms * 1e-3),
            "frac_literal": max(useful / (peaks["bf16_tflops"] * 1e12), t_hbm) / (spmm_ms * 1e-3)}


def all_cells():
    """Every (config, layer, N:M, keep) the metric names: config 1, config 2, the 13 VGG-16 and the 35
    MobileNetV2 layers, the 5 x 4 sweep, and 3:4 on the sweep shape."""
    return wl.config1() + wl.config2() + wl.config3() + wl.config4() + wl.config5() + wl.extra_sweep_cells()


def device_activation(torch, layer, dev):
    """X[k, ncols] bf16 drawn on the device (N(0,1), rectified for the network layers): the stand-in for the
    layer's input activations.  Same distribution as workloads.make_activation; the large layers' X (up to
    0.9 GB) is not worth a host draw and a copy per cell."""
    g = torch.Generator(device=dev)
    g.manual_seed(layer.seed + 7)
    x = torch.randn((layer.k, layer.ncols), device=dev, generator=g)
    if layer.relu_x:
        x.clamp_(min=0)
    return x.to(torch.bfloat16)


def measure_cells(torch, B, dev, peaks, flush_l2, shared, iters=50):
    """SpMM-only timing of every cell of the metric, each beside a dense bf16 cuBLAS GEMM of the same shape.
    Cold L2: `iters` launches, each after an L2 flush, each in its own event pair (median and minimum).
    Warm L2: the same launch repeated back to back on the same buffers, `iters` launches in five event pairs
    (median and minimum of the five averages); for layers larger than L2 that is simply a pipelined stream of
    launches.  (measure_cells_graph adds a third protocol to the same records.)"""
    out = []
    stream = torch.cuda.current_stream()

    def cold(fn):
        ts = []
        for i in range(3 + iters):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        return float(np.median(ts)), float(np.min(ts))

    def warm(fn):
        per = max(1, iters // 5)
        ts = []
        for _ in range(3):
            fn()
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(per):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3 / per)
        return float(np.median(ts)), float(np.min(ts))

    for layer in all_cells():
        if layer.config == 5:
            d_s, d_w, d_x = shared                      # every sweep cell prunes the same W / S / X
        else:
            w = wl.make_weight(layer)
            d_s = torch.from_numpy(wl.make_saliency(layer, w)).to(dev)
            d_w = torch.from_numpy(w.view(np.int16)).to(dev).view(torch.bfloat16)
            d_x = device_activation(torch, layer, dev)
        d_y = torch.empty((layer.rows, layer.ncols), dtype=torch.bfloat16, device=dev)
        L = B.HybridLayer(layer.rows, layer.k, layer.n, layer.m, layer.block_rows, layer.block_k,
                          layer.keep_ratio, device=dev)
        L.build_mask(d_s).encode(d_w)
        ours = lambda: L.spmm(d_x, y=d_y)
        dense = lambda: torch.matmul(d_w, d_x, out=d_y)
        c_med, c_min = cold(ours)
        w_med, w_min = warm(ours)
        launched = L.last_launch()
        dc_med, dc_min = cold(dense)
        dw_med, dw_min = warm(dense)
        model = L.bytes_model(layer.ncols)
        rec = {"workload": layer.name, "config": layer.config, "rows": layer.rows, "k": layer.k,
               "ncols": layer.ncols, "nm": f"{layer.n}:{layer.m}", "block": [layer.block_rows, layer.block_k],
               "keep": round(layer.keep_ratio, 4), "kkeep": L.kkeep, "kernel": B.PATH_NAMES[launched["path"]],
               "tile_cols": launched["tile_cols"], "accumulators": launched["accumulators"],
               "stack": launched["stack"], "stage_blocks": launched["stage_blocks"],
               "spmm_us": c_med, "spmm_us_min": c_min, "spmm_warm_us": w_med, "spmm_warm_us_min": w_min,
               "dense_cublas_us": dc_med, "dense_cublas_us_min": dc_min, "dense_cublas_warm_us": dw_med,
               "speedup_vs_dense_cublas": dc_med / c_med, "speedup_warm": dw_med / w_med,
               "device_status": L.device_status()}
        if L.kkeep > 0:
            r = roofline_terms(model, peaks, c_med * 1e-3, layer.ncols)
            rec.update({"useful_tflops": r["useful_flops"] / (c_med * 1e-6) / 1e12,
                        "t_tensor_us": r["t_tensor"] * 1e6, "t_hbm_us": r["t_hbm"] * 1e6,
                        "roofline_frac": r["frac"], "roofline_frac_literal": r["frac_literal"],
                        "roofline_frac_warm": r["frac"] * c_med / w_med})
        else:
            # no kept block (a one-block layer below keep 0.5): Y = 0, no useful work, kept out of the sums
            rec.update({"useful_tflops": 0.0, "roofline_frac": None, "roofline_frac_literal": None})
        out.append(rec)
        L.close()
        del d_y
        if layer.config != 5:
            del d_x, d_w, d_s
    return out


def measure_cells_graph(torch, B, dev, shared, cells):
    """Graph replay of every cell, added to the records of measure_cells: 20 launches captured in a CUDA graph and
    replayed (median and minimum per launch over 9 replays), ours and the dense cuBLAS GEMM: device time without
    the host's launch path and without the 2 us tick of the event timer, which is what separates layers of a few
    microseconds; operands stay in L2 where they fit.  A pass of its own, after every other figure of the run
    has been taken: the replays keep the GPU under load for seconds, and cold launches measured in between came
    out up to 20 % slower (ours and cuBLAS alike)."""
    side = torch.cuda.Stream()

    def replay(fn, n=20, reps=9):
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            fn(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for _ in range(n):
                    fn(side)
            g.replay()
            torch.cuda.synchronize()
            ts = []
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(side); g.replay(); b.record(side)
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b) * 1e3 / n)
        del g
        return float(np.median(ts)), float(np.min(ts))

    for rec, layer in zip(cells, all_cells()):
        if layer.config == 5:
            d_s, d_w, d_x = shared
        else:
            w = wl.make_weight(layer)
            d_s = torch.from_numpy(wl.make_saliency(layer, w)).to(dev)
            d_w = torch.from_numpy(w.view(np.int16)).to(dev).view(torch.bfloat16)
            d_x = device_activation(torch, layer, dev)
        d_y = torch.empty((layer.rows, layer.ncols), dtype=torch.bfloat16, device=dev)
        L = B.HybridLayer(layer.rows, layer.k, layer.n, layer.m, layer.block_rows, layer.block_k,
                          layer.keep_ratio, device=dev)
        L.build_mask(d_s).encode(d_w)
        g_med, g_min = replay(lambda st: L.spmm(d_x, y=d_y, stream=st))
        dg_med, dg_min = replay(lambda st: torch.matmul(d_w, d_x, out=d_y))
        rec.update({"spmm_graph_us": g_med, "spmm_graph_us_min": g_min, "dense_cublas_graph_us": dg_med,
                    "dense_cublas_graph_us_min": dg_min, "speedup_graph": dg_med / g_med})
        if L.device_status() != 0:
            rec["device_status"] = L.device_status()
        L.close()
        del d_y
        if layer.config != 5:
            del d_x, d_w, d_s
    return cells


def measure_two_addends(torch, B, dev, peaks, flush_l2, shared, iters=30):
    """Patterns 2:4 cannot express in one pass (3:4, 4:8): the dense-tile image (default) against the same block
    split into two 2:4-compliant addends that are multiplied into one accumulator by two sparse passes over the
    same X tile.  Same tensor slots either way; the two-addend form moves 20 KB instead of 16 KB of weights per
    block and, with 256-column tiles, has room for one accumulator only."""
    d_s, d_w, d_x = shared
    stream = torch.cuda.current_stream()
    out = []
    for (n, m, keep) in ((4, 8, 0.5), (4, 8, 0.25), (3, 4, 0.5), (3, 4, 0.25)):
        layer = wl.sweep_cell(n, m, keep)
        d_y = torch.empty((layer.rows, layer.ncols), dtype=torch.bfloat16, device=dev)
        rec = {"workload": layer.name}
        ys = {}
        for kind in ("dense", "sparse2"):
            os.environ["CRISP_EXEC_IMAGE"] = kind
            L = B.HybridLayer(layer.rows, layer.k, n, m, layer.block_rows, layer.block_k, keep, device=dev)
            L.build_mask(d_s).encode(d_w)
            os.environ.pop("CRISP_EXEC_IMAGE")
            ts = []
            for i in range(3 + iters):
                flush_l2()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); L.spmm(d_x, y=d_y); b.record(stream)
                torch.cuda.synchronize()
                if i >= 3:
                    ts.append(a.elapsed_time(b) * 1e3)
            ys[kind] = d_y.clone()
            r = roofline_terms(L.bytes_model(layer.ncols), peaks, float(np.median(ts)) * 1e-3, layer.ncols)
            rec[kind] = {"kernel": B.PATH_NAMES[L.last_launch()["path"]], "spmm_us": float(np.median(ts)),
                         "spmm_us_min": float(np.min(ts)), "roofline_frac": r["frac"], "device_status": L.device_status()}
            L.close()
        d = (ys["dense"].float() - ys["sparse2"].float()).abs().max().item()
        rec["max_abs_difference"] = d
        rec["two_addends_over_dense"] = rec["sparse2"]["spmm_us"] / rec["dense"]["spmm_us"]
        out.append(rec)
    return out


def summarise_cells(cells):
    """Per workload family: sum of our times, sum of the dense cuBLAS times, their ratio (layers with no kept
    block left out), and the spread of the roofline fraction."""
    fam = {1: "config1", 2: "config2_resnet50_layer3", 3: "config3_vgg16", 4: "config4_mobilenetv2", 5: "config5_sweep"}
    out = {}
    for cfg, name in fam.items():
        cs = [c for c in cells if c["config"] == cfg and c["kkeep"] > 0]
        if not cs:
            continue
        ours, dense = sum(c["spmm_us"] for c in cs), sum(c["dense_cublas_us"] for c in cs)
        g_ours, g_dense = sum(c["spmm_graph_us"] for c in cs), sum(c["dense_cublas_graph_us"] for c in cs)
        fr = [c["roofline_frac"] for c in cs]
        out[name] = {"layers": len(cs), "spmm_us_sum": ours, "dense_cublas_us_sum": dense,
                     "speedup_vs_dense_cublas": dense / ours,
                     "spmm_graph_us_sum": g_ours, "dense_cublas_graph_us_sum": g_dense, "speedup_graph": g_dense / g_ours,
                     "faster_than_dense_graph": sum(1 for c in cs if c["speedup_graph"] >= 1.0),
                     "useful_tflops": sum(c["useful_tflops"] * c["spmm_us"] for c in cs) / ours,
                     "roofline_frac_min": min(fr), "roofline_frac_median": float(np.median(fr)),
                     "roofline_frac_max": max(fr),
                     "faster_than_dense": sum(1 for c in cs if c["speedup_vs_dense_cublas"] >= 1.0)}
    low = [c for c in cells if c["config"] == 5 and c["keep"] <= 0.5 and c["kkeep"] > 0]
    out["sweep_keep_le_0.5"] = {"cells": len(low),
                                "at_or_above_60pct_of_roofline": sum(1 for c in low if c["roofline_frac"] >= 0.6),
                                "faster_than_dense": sum(1 for c in low if c["speedup_vs_dense_cublas"] >= 1.0)}
    return out


def measure_global_rank(torch, B, dev, with_oracle, iters=12):
    """Global rank selection (Algorithm 1: per-row sort, rank-column sums, global order, selection by the
    sparsity target) over the VGG-16 and MobileNetV2 stand-in networks: device time of crisp_global_rank
    on the block scores that crisp_build_mask left on the device, and the oracle's time for the same step."""
    out = []
    stream = torch.cuda.current_stream()
    for name, cfg in (("vgg16", wl.config3()), ("mobilenetv2", wl.config4())):
        layers, sal = [], []
        for l in cfg:
            s = wl.make_saliency(l, wl.make_weight(l))
            L = B.HybridLayer(l.rows, l.k, l.n, l.m, l.block_rows, l.block_k, 1.0, device=dev)
            L.build_mask(torch.from_numpy(s).to(dev))
            layers.append(L); sal.append(s)
        arr = B.make_rank_layers([L.rank_layer(1) for L in layers])
        ws = torch.empty(B.crisp_global_rank_sizes(arr), dtype=torch.uint8, device=dev)
        kk = torch.zeros(len(layers), dtype=torch.int32, device=dev)
        ts = []
        for i in range(3 + iters):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            B.crisp_global_rank(arr, 0.6, ws, kk)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        rec = {"network": name, "layers": len(layers), "rank_positions": int(sum(L.nblk - 1 for L in layers)),
               "block_scores": int(sum(L.nrt * L.nblk for L in layers)), "prune_fraction": 0.6,
               "global_rank_us": float(np.mean(ts)) * 1e3, "launches": 3,
               "kkeep": kk.cpu().numpy().tolist()}
        if with_oracle:
            import oracle
            import time
            scores = []
            for L in layers:
                sc_ptr, _ = B.crisp_mask_scores(L.desc, L.workspace)
                off = sc_ptr - L.workspace.data_ptr()
                scores.append(L.workspace[off: off + 8 * L.nrt * L.nblk].view(torch.int64).cpu().numpy()
                              .view(np.uint64).reshape(L.nrt, L.nblk))
            exps = [oracle.score_scale_exp(s) for s in sal]
            elems = [L.desc.block_rows * L.desc.block_k for L in layers]
            t0 = time.perf_counter()
            want = oracle.global_rank(scores, exps, elems, 0.6, min_keep=[1] * len(layers))
            rec["oracle_us"] = (time.perf_counter() - t0) * 1e6
            rec["matches_oracle"] = bool(np.array_equal(want, np.array(rec["kkeep"])))
        for L in layers:
            L.close()
        out.append(rec)
    return out


def measure_iteration(torch, B, dev, with_oracle, samples=4, iters=9):
    """One pruning iteration of Algorithm 1 over a whole network without the fine-tuning (saliency of Eq. 1 from
    `samples` bf16 gradient tensors per layer, N:M step + block scores, global rank selection, per-row-tile
    selection, compression), through binding.PruningNetwork: device time of the whole sequence (it contains one
    small device-to-host read of the selected counts), its launches, and the oracle's time for the same step."""
    out = []
    stream = torch.cuda.current_stream()
    for name, cfg in (("vgg16", wl.config3()), ("mobilenetv2", wl.config4())):
        n, m, bm, bk = cfg[0].n, cfg[0].m, cfg[0].block_rows, cfg[0].block_k
        shapes = [(l.rows, l.k) for l in cfg]
        w_host = [wl.make_weight(l) for l in cfg]
        g = torch.Generator(device=dev); g.manual_seed(cfg[0].seed + 91)
        d_w = [torch.from_numpy(w.view(np.int16)).to(dev).view(torch.bfloat16) for w in w_host]
        d_g = [[(torch.randn(sh, device=dev, generator=g) * 1e-2).to(torch.bfloat16) for _ in range(samples)] for sh in shapes]
        net = B.PruningNetwork(shapes, n, m, bm, bk, min_keep=1, device=dev)
        kappa = 1.0 - 0.5 * n / m                                 # half of the blocks of the network
        ts = []
        for i in range(3 + iters):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            kk = net.step(d_w, d_g, kappa)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        weights = sum(r * k for r, k in shapes)
        rec = {"network": name, "layers": len(shapes), "weights": int(weights), "samples": samples, "kappa": kappa,
               "iteration_us": float(np.median(ts)), "iteration_us_min": float(np.min(ts)),
               "launches": len(shapes) * (samples + 2 + 3 + 1 + 2) + 3, "kkeep": [int(c) for c in kk],
               "algorithmic_bytes": int(weights * (samples * 2 + (samples - 1) * 8 + 4 + 2 + 4 + 4 + 4 + 2 + 2))}
        rec["achieved_gbs"] = rec["algorithmic_bytes"] / (rec["iteration_us"] * 1e-6) / 1e9
        if with_oracle:
            import oracle
            grads = [np.stack([wl.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16)) for t in gs]) for gs in d_g]
            t0 = time.perf_counter()
            sal = [oracle.saliency_f32(gr, w) for gr, w in zip(grads, w_host)]
            full = [oracle.build_mask(s_, n, m, bm, bk, 1.0) for s_ in sal]
            want = oracle.global_rank([f.score for f in full], [oracle.score_scale_exp(s_) for s_ in sal],
                                      [bm * bk] * len(full), B.crisp_prune_fraction(kappa, n, m), min_keep=[1] * len(full))
            for s_, w, f, c in zip(sal, w_host, full, want):
                oracle.encode(w, oracle.build_mask(s_, n, m, bm, bk, float(c) / f.nblk))
            rec["oracle_us"] = (time.perf_counter() - t0) * 1e6
            rec["matches_oracle"] = bool([int(c) for c in want] == rec["kkeep"])
        net.close()
        out.append(rec)
    return out


_VGG_CONV = {1: (64, 224), 2: (64, 112), 3: (128, 112)}     # config-3 layer index -> (input channels, side)


def measure_conv(torch, B, dev, peaks, flush_l2, iters=9):
    """Convolution as implicit GEMM (crisp_spmm_conv on the NHWC activation) beside the same layer run as
    crisp_spmm on the lowered K x Nc matrix and beside dense cuBLAS on that matrix: the three largest VGG-16
    layers of config 3 (batch 16).  Roofline terms of the implicit call: the activation is read once."""
    out = []
    stream = torch.cuda.current_stream()

    def timed(fn):
        ts = []
        for i in range(3 + iters):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        return float(np.mean(ts))

    cfg = wl.config3()
    for idx, (cin, side) in _VGG_CONV.items():
        layer, batch = cfg[idx], 16
        w = wl.make_weight(layer)
        s = wl.make_saliency(layer, w)
        d_w = torch.from_numpy(w.view(np.int16)).to(dev).view(torch.bfloat16)
        g = torch.Generator(device=dev); g.manual_seed(layer.seed + 7)
        act = torch.randn((batch, side, side, cin), device=dev, generator=g).clamp_(min=0).to(torch.bfloat16)
        L = B.HybridLayer(layer.rows, layer.k, layer.n, layer.m, layer.block_rows, layer.block_k, layer.keep_ratio,
                          device=dev)
        L.build_mask(torch.from_numpy(s).to(dev)).encode(d_w)
        ncols = batch * side * side
        y = torch.empty((layer.rows, ncols), dtype=torch.bfloat16, device=dev)
        y2 = torch.empty_like(y)
        ms_i = timed(lambda: L.spmm_conv(act, 3, 3, 1, y=y))
        ap = torch.nn.functional.pad(act, (0, 0, 1, 1, 1, 1))
        x = torch.stack([ap[:, i:i + side, j:j + side, :] for i in range(3) for j in range(3)], dim=0) \
            .permute(0, 4, 1, 2, 3).reshape(9 * cin, ncols).contiguous()
        del ap
        ms_e = timed(lambda: L.spmm(x, y=y2))
        ms_d = timed(lambda: torch.matmul(d_w, x, out=y2))
        L.spmm(x, y=y2)
        torch.cuda.synchronize()
        m = L.bytes_model(ncols)
        alg = m["vals_bytes"] + m["idx_bytes"] + m["blk_col_bytes"] + act.numel() * 2 + m["y_bytes"]
        t_hbm = alg / (peaks["hbm_gbs"] * 1e9)
        r = roofline_terms(m, peaks, ms_i, ncols)
        out.append({"workload": layer.name, "activation": [batch, side, side, cin], "kkeep": L.kkeep,
                    "conv_us": ms_i * 1e3, "lowered_spmm_us": ms_e * 1e3, "dense_cublas_lowered_us": ms_d * 1e3,
                    "speedup_vs_lowered": ms_e / ms_i, "speedup_vs_dense_cublas": ms_d / ms_i,
                    "algorithmic_bytes": int(alg), "t_hbm_us": t_hbm * 1e6, "t_tensor_us": r["t_tensor"] * 1e6,
                    "roofline_frac": max(t_hbm, r["t_tensor"]) / (ms_i * 1e-3),
                    "identical_to_lowered": bool(torch.equal(y, y2)), "device_status": L.device_status()})
        L.close()
        del x, y, y2, act
    return out


def measure_saliency(torch, B, dev, peaks, flush_l2, shared, samples=4, iters=9):
    """Saliency score of Eq. 1 on the sweep layer (4096 x 4096): `samples` gradient tensors (bf16) accumulated,
    then S = |mean g * W|.  HBM roofline: per accumulate 2 + 4 (+ 4 after the first) bytes per weight, per
    finish 4 + 2 + 4."""
    _d_s, d_w, _d_x = shared
    rows, k = d_w.shape
    stream = torch.cuda.current_stream()
    g = torch.Generator(device=dev); g.manual_seed(77)
    grads = [(torch.randn((rows, k), device=dev, generator=g) * 1e-2).to(torch.bfloat16) for _ in range(samples)]
    acc = torch.empty((rows, k), dtype=torch.float32, device=dev)
    s = torch.empty((rows, k), dtype=torch.float32, device=dev)
    ts = []
    for i in range(3 + iters):
        flush_l2()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for j, gr in enumerate(grads):
            B.crisp_saliency_accumulate(gr, 0, k, rows, k, acc, k, j == 0)
        B.crisp_saliency_finish(acc, k, d_w, k, rows, k, samples, s, k)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            ts.append(a.elapsed_time(b))
    ms = float(np.mean(ts))
    n = rows * k
    alg = n * (6 + (samples - 1) * 10 + 10)
    return {"workload": f"saliency_{rows}x{k}_{samples}samples_bf16grad", "us": ms * 1e3, "launches": samples + 1,
            "algorithmic_bytes": int(alg), "achieved_gbs": alg / (ms * 1e-3) / 1e9,
            "roofline_frac": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}


def recorded_traffic(workload, kernel):
    """DRAM bytes per launch from the committed ncu capture, or None when the kernel source has
    changed since the counters were taken."""
    import hashlib
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return None
    rec = json.load(open(p))
    src = os.path.join(ROOT, "paper_2311_14272_b200", "csrc", "spmm_tc.cu")
    sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
    for r in rec.get("captures", []):
        if r["workload"] == workload and r["kernel"] == kernel and r["source_sha256"] == sha:
            return r["dram_bytes_per_launch"]
    return None


def max_over_ranks(torch, value, world, device):
    """The largest `value` over the ranks of the job: the slowest rank's time is the job's time."""
    t = torch.tensor([value], device=device, dtype=torch.float64)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank_step, world, ms_per_step):
    """The path does not shard: N ranks are N replicas, each with the whole layer on its own inputs (weak scaling,
    no data-path collective).  The job's throughput is all ranks' work over the slowest rank's step time."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def run_ours(args, layer, rank, world):
    import torch
    import torch.distributed as dist
    from paper_2311_14272_b200 import binding as B

    B.load()                                       # raises if libcrisp.so is missing: no fallback
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks, peak_kind = load_peaks()

    w, s, x = wl.make_layer_inputs(layer)
    h_s = torch.from_numpy(s).pin_memory()
    h_w = torch.from_numpy(w.view(np.int16)).pin_memory()
    h_x = torch.from_numpy(x.view(np.int16)).pin_memory()
    d_s = h_s.to(dev)
    d_w = h_w.to(dev).view(torch.bfloat16)
    d_x = h_x.to(dev).view(torch.bfloat16)
    d_y = torch.empty((layer.rows, layer.ncols), dtype=torch.bfloat16, device=dev)
    h_y = torch.empty((layer.rows, layer.ncols), dtype=torch.bfloat16).pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_sink = torch.zeros(1, dtype=torch.int64, device=dev)
    L = B.HybridLayer(layer.rows, layer.k, layer.n, layer.m, layer.block_rows, layer.block_k,
                      layer.keep_ratio, device=dev)
    stream = torch.cuda.current_stream()

    def flush_l2():
        # overwrite 256 MiB (evicts everything), then read it back so that the lines left in L2 are
        # clean: otherwise the write-back of ~126 MB of dirty lines is charged to the next kernels
        flush.zero_()
        flush_sink.copy_(flush.view(torch.int64).max().view(1))

    def step():
        L.build_mask(d_s)
        L.encode(d_w)
        L.spmm(d_x, y=d_y)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        flush_l2()
        step()
    torch.cuda.synchronize()
    if L.device_status() != 0:
        raise SystemExit(f"device status {L.device_status()} after warm-up")
    model = L.bytes_model(layer.ncols)
    nnz = model["nnz"]

    # ---- timed region: K steps, each bracketed by events on the launching stream; L2 is flushed
    # between steps (outside the event pairs) by overwriting a 256 MiB buffer
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    barrier()
    sampler.start()
    # The host must never be what a timed event pair waits for (a busy host, or this process's own sampling thread,
    # can take longer to queue a launch than the GPU takes to run the previous one).  So some 15 ms of untimed fills
    # go in first: while the GPU works through them the host queues every timed step, and the steps then run back
    # to back off the stream's queue.
    for _ in range(200):
        flush.zero_()
    for i in range(args.steps):
        flush_l2()
        ev[i][0].record(stream)
        L.build_mask(d_s)
        ev[i][1].record(stream)
        L.encode(d_w)
        ev[i][2].record(stream)
        L.spmm(d_x, y=d_y)
        ev[i][3].record(stream)
    while not ev[-1][3].query():                   # the sampling thread runs while the GPU works through the queue
        sampler.sample()
        time.sleep(0.0005)
    barrier()
    clocks = sampler.stop()
    t_mask = np.array([e[0].elapsed_time(e[1]) for e in ev])
    t_enc = np.array([e[1].elapsed_time(e[2]) for e in ev])
    t_spmm = np.array([e[2].elapsed_time(e[3]) for e in ev])
    t_step = np.array([e[0].elapsed_time(e[3]) for e in ev])
    ms_local = float(t_step.sum() / args.steps)
    ms_per_step = max_over_ranks(torch, ms_local, world, dev)
    status = L.device_status()

    # ---- dense bf16 cuBLAS GEMM of the same shape, same protocol
    evd = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(3 + args.steps)]
    for _ in range(100):                           # queued behind untimed fills, like the steps above
        flush.zero_()
    for a, b in evd:
        flush_l2()
        a.record(stream)
        torch.matmul(d_w, d_x, out=d_y)
        b.record(stream)
    torch.cuda.synchronize()
    t_dense = np.array([a.elapsed_time(b) for a, b in evd[3:]])

    # ---- end to end: pinned host inputs -> device, whole path, result back to pinned host memory.
    # Every step copies its own S, W and X from pinned host memory and its Y back; two sets of device
    # buffers and two copy streams let the copies of step i+1 run while step i computes and reads back
    # (PCIe is full duplex), as a caller that streams layers through the library would do.  The same
    # loop on one stream (no overlap) is reported beside it.
    def e2e_step():
        d_s.copy_(h_s, non_blocking=True)
        d_w.view(torch.int16).copy_(h_w, non_blocking=True)
        d_x.view(torch.int16).copy_(h_x, non_blocking=True)
        step()
        h_y.copy_(d_y, non_blocking=True)

    d_in = [(d_s, d_w, d_x), (torch.empty_like(d_s), torch.empty_like(d_w), torch.empty_like(d_x))]
    d_out = [d_y, torch.empty_like(d_y)]
    h_out = [h_y, torch.empty((layer.rows, layer.ncols), dtype=torch.bfloat16).pin_memory()]
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_cmp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_pipelined(n, start_event):
        s_in.wait_event(start_event)
        for it in range(n):
            k = it & 1
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_cmp[k])               # the step that last read this buffer set is done
                d_in[k][0].copy_(h_s, non_blocking=True)
                d_in[k][1].view(torch.int16).copy_(h_w, non_blocking=True)
                d_in[k][2].view(torch.int16).copy_(h_x, non_blocking=True)
                ev_in[k].record(s_in)
            stream.wait_event(ev_in[k])
            stream.wait_event(ev_out[k])                 # this Y buffer has been read back
            L.build_mask(d_in[k][0])
            L.encode(d_in[k][1])
            L.spmm(d_in[k][2], y=d_out[k])
            ev_cmp[k].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[k])
                h_out[k].copy_(d_out[k], non_blocking=True)
                ev_out[k].record(s_out)
        stream.wait_event(ev_out[0])
        stream.wait_event(ev_out[1])

    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        e2e_step()
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    b.record(stream)
    barrier()
    e2e_serial_ms = a.elapsed_time(b) / e2e_steps
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    e2e_pipelined(2, a)
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    e2e_pipelined(e2e_steps, a)
    b.record(stream)
    barrier()
    if not torch.equal(h_out[0], h_out[1]):
        raise SystemExit("end-to-end pipeline: the two result buffers differ")
    e2e_ms = max_over_ranks(torch, a.elapsed_time(b) / e2e_steps, world, dev)

    # ---- end to end, inference style: the handle (mask + encoding) is reused, a step is X in -> product -> Y out.
    # Same pipelining: the copy of the next X and the read-back of the previous Y overlap the product.
    def inf_pipelined(n, start_event):
        s_in.wait_event(start_event)
        for it in range(n):
            k = it & 1
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_cmp[k])
                d_in[k][2].view(torch.int16).copy_(h_x, non_blocking=True)
                ev_in[k].record(s_in)
            stream.wait_event(ev_in[k])
            stream.wait_event(ev_out[k])
            L.spmm(d_in[k][2], y=d_out[k])
            ev_cmp[k].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[k])
                h_out[k].copy_(d_out[k], non_blocking=True)
                ev_out[k].record(s_out)
        stream.wait_event(ev_out[0])
        stream.wait_event(ev_out[1])

    L.build_mask(d_s)
    L.encode(d_w)
    a = torch.cuda.Event(enable_timing=True)
    a.record(stream)
    inf_pipelined(2, a)
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    inf_pipelined(e2e_steps, a)
    b.record(stream)
    barrier()
    inf_ms = max_over_ranks(torch, a.elapsed_time(b) / e2e_steps, world, dev)

    # ---- the SpMM kernel as a stream of launches: back to back on three rotating sets of X / Y (384 MB, larger
    # than L2, so every launch finds its operands in HBM), one event pair around the whole stream
    xs = [d_x, d_in[1][2], torch.empty_like(d_x)]
    xs[1].copy_(d_x); xs[2].copy_(d_x)
    ys = [d_y, d_out[1], torch.empty_like(d_y)]
    b2b = []
    for rep in range(4):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_launch = 18
        a.record(stream)
        for i in range(n_launch):
            L.spmm(xs[i % 3], y=ys[i % 3])
        b.record(stream)
        torch.cuda.synchronize()
        if rep:
            b2b.append(a.elapsed_time(b) * 1e3 / n_launch)
    t_b2b_us = float(np.median(b2b))
    del xs, ys

    useful_flops = 2.0 * nnz * layer.ncols
    value = whole_job_tflops(useful_flops, world, ms_per_step)
    e2e_value = whole_job_tflops(useful_flops, world, e2e_ms)

    # ---- roofline of the dominant kernel (SpMM), from its live event time
    spmm_ms = float(t_spmm.mean())
    slot_flops = 2.0 * model["slot_macs"]
    hbm_bytes = model["vals_bytes"] + model["idx_bytes"] + model["blk_col_bytes"] + model["x_bytes"] + model["y_bytes"]
    t_tensor = slot_flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = hbm_bytes / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        roof = {"bound": "tensor", "achieved": slot_flops / (spmm_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": hbm_bytes / (spmm_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    launched = L.last_launch()
    roof.update({"traffic": recorded_traffic(args.workload, B.PATH_NAMES[launched["path"]]), "peak_kind": f"of {peak_kind} (burst)",
                 "kernel": B.PATH_NAMES[launched["path"]], "tile_cols": launched["tile_cols"],
                 "accumulators": launched["accumulators"], "ring_stages": launched["stages"], "ctas": launched["ctas"],
                 "t_tensor_us": t_tensor * 1e6, "t_hbm_us": t_hbm * 1e6, "t_kernel_us": spmm_ms * 1e3,
                 "t_kernel_median_us": float(np.median(t_spmm) * 1e3), "t_kernel_min_us": float(t_spmm.min() * 1e3),
                 "t_kernel_timing": "mean over the timed steps of the event pair around the crisp_spmm launch (L2 flushed before every step)",
                 "t_kernel_back_to_back_us": t_b2b_us,
                 "frac_back_to_back": max(t_tensor, t_hbm) / (t_b2b_us * 1e-6),
                 "dense_cublas_us": float(t_dense.mean() * 1e3),
                 "speedup_vs_dense_cublas": float(t_dense.mean() / t_spmm.mean()),
                 "frac_of_max_roof": max(t_tensor, t_hbm) / (spmm_ms * 1e-3),
                 "frac_literal_useful_flops": useful_flops / (spmm_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                 "algorithmic_bytes": hbm_bytes, "slot_flops": slot_flops})
    mask_bytes = layer.rows * layer.k * 4 * 2 + layer.rows * layer.k // 8   # S read twice (max, select) + bits
    enc_bytes = model["vals_bytes"] * 2 + model["idx_bytes"] + layer.rows * layer.k // 8
    phases = {"mask_us": float(t_mask.mean() * 1e3), "encode_us": float(t_enc.mean() * 1e3),
              "spmm_us": spmm_ms * 1e3, "spmm_us_min": float(t_spmm.min() * 1e3),
              "mask_gbs": mask_bytes / (t_mask.mean() * 1e-3) / 1e9,
              "encode_gbs": enc_bytes / (t_enc.mean() * 1e-3) / 1e9,
              "spmm_useful_tflops": useful_flops / (spmm_ms * 1e-3) / 1e12,
              "dense_cublas_us": float(t_dense.mean() * 1e3),
              "spmm_speedup_vs_dense_cublas": float(t_dense.mean() / t_spmm.mean())}

    # mask: max_key, group_select, block_select; encode: encode_block (+ tiles for 128-row blocks), walk lists,
    # and a separate image kernel for narrower blocks; spmm: one persistent kernel
    kernels_per_step = {"mask": 3, "encode": 1 if layer.block_rows == 128 else 2, "spmm": 1}
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": args.workload, "rows": layer.rows, "k": layer.k, "ncols": layer.ncols,
                      "n": layer.n, "m": layer.m, "block": [layer.block_rows, layer.block_k],
                      "keep_ratio": layer.keep_ratio, "kkeep": L.kkeep, "nnz": nnz,
                      "step": "crisp_build_mask + crisp_encode + crisp_spmm",
                      "l2": "flushed between steps (256 MiB overwritten, then read back, outside the event pairs)",
                      "parallelism": "replicas only" if world > 1 else "single GPU"},
           "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "serial_ms_per_step": e2e_serial_ms,
                   "overlap": "copies of step i+1 overlap compute and read-back of step i (2 buffer sets, 3 streams)",
                   "h2d_bytes_per_step": int(h_s.numel() * 4 + h_w.numel() * 2 + h_x.numel() * 2),
                   "d2h_bytes_per_step": int(h_y.numel() * 2)},
           "e2e_inference": {"value": whole_job_tflops(useful_flops, world, inf_ms), "unit": UNIT, "ms_per_step": inf_ms,
                             "step": "X host -> device, crisp_spmm on the resident handle, Y device -> host (2 buffer sets, 3 streams)",
                             "h2d_bytes_per_step": int(h_x.numel() * 2), "d2h_bytes_per_step": int(h_y.numel() * 2)},
           "gpu_launches": sum(kernels_per_step.values()) * args.steps, "kernels_per_step": kernels_per_step,
           "clocks": clocks, "roofline": roof, "phases": phases, "device_status": status}

    if rank == 0 and world == 1 and not args.no_cells and args.workload.startswith("sweep_"):
        cells = measure_cells(torch, B, dev, peaks, flush_l2, (d_s, d_w, d_x), iters=args.cell_iters)
        out["cells"] = cells
        out["global_rank"] = measure_global_rank(torch, B, dev, not args.no_cpu_baseline)
        out["conv"] = measure_conv(torch, B, dev, peaks, flush_l2)
        out["saliency"] = measure_saliency(torch, B, dev, peaks, flush_l2, (d_s, d_w, d_x))
        out["pruning_iteration"] = measure_iteration(torch, B, dev, not args.no_cpu_baseline)
        out["two_addend_form"] = measure_two_addends(torch, B, dev, peaks, flush_l2, (d_s, d_w, d_x))
        measure_cells_graph(torch, B, dev, (d_s, d_w, d_x), cells)
        out["summary"] = summarise_cells(cells)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        cols = oracle_sample_cols(layer, w, s, x)
        dt, onnz = oracle_step(layer, w, s, np.ascontiguousarray(x[:, :cols]))
        out["cpu_baseline"] = {"value": 2.0 * onnz * cols / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
                               "kind": "oracle", "seconds": dt,
                               "sample": f"mask+encode+decode of the full layer, fp64 product on the first {cols} "
                                         f"of {layer.ncols} columns"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def render_markdown(d):
    """Markdown tables of one JSON line of this program (the repository's table of measured numbers is this output)."""
    o = []
    r, ph, c = d["roofline"], d["phases"], d["config"]
    o.append(f"Headline step ({c['workload']}, {c['rows']}x{c['k']}x{c['ncols']}, block {c['block'][0]}x{c['block'][1]}, "
             f"kkeep {c['kkeep']}): `value` {d['value']:.1f} useful TFLOP/s, `ms_per_step` {d['ms_per_step'] * 1e3:.1f} us "
             f"(`phases`: mask {ph['mask_us']:.1f}, encode {ph['encode_us']:.1f}, SpMM {ph['spmm_us']:.1f} us; "
             f"{d['steps']} steps, L2 flushed before each).")
    o.append(f"`roofline`: bound {r['bound']}, kernel {r['kernel']}, `t_kernel_us` {r['t_kernel_us']:.1f} (median "
             f"{r['t_kernel_median_us']:.1f}, min {r['t_kernel_min_us']:.1f}; back to back {r['t_kernel_back_to_back_us']:.1f}), "
             f"`t_tensor_us` {r['t_tensor_us']:.1f}, `t_hbm_us` {r['t_hbm_us']:.1f}, `frac` {r['frac']:.3f} "
             f"(back to back {r['frac_back_to_back']:.3f}) {r['peak_kind']}, `speedup_vs_dense_cublas` "
             f"{r['speedup_vs_dense_cublas']:.2f} (dense {r['dense_cublas_us']:.1f} us), `traffic` {r['traffic']}.")
    e, ei = d["e2e"], d["e2e_inference"]
    o.append(f"`e2e` (S, W, X in and Y out every step): {e['ms_per_step']:.2f} ms, {e['value']:.1f} TFLOP/s "
             f"(one stream: {e['serial_ms_per_step']:.2f} ms); `e2e_inference` (handle resident, X in, Y out): "
             f"{ei['ms_per_step']:.2f} ms, {ei['value']:.1f} TFLOP/s.")
    if "cpu_baseline" in d:
        cb = d["cpu_baseline"]
        o.append(f"`cpu_baseline` (oracle, {cb['cores']} host cores, {cb['sample']}): {cb['value']:.4f} TFLOP/s.")
    cells = d.get("cells", [])

    def row(x):
        fr = "-" if x["roofline_frac"] is None else f"{x['roofline_frac']:.2f} / {x['roofline_frac_literal']:.2f}"
        return (f"| {x['workload']} | {x['rows']}x{x['k']}x{x['ncols']} | {x['nm']} | {x['kkeep']} | {x['kernel'].replace('_tcgen05', '')} "
                f"{x['tile_cols']}c/{x['accumulators']}a{'/s' + str(x['stack']) if x['stack'] > 1 else ''}"
                f"{'/b' + str(x['stage_blocks']) if x.get('stage_blocks', 1) > 1 else ''} | {x['spmm_us']:.1f} ({x['spmm_us_min']:.1f}) | "
                f"{x['spmm_warm_us']:.1f} | {x['dense_cublas_us']:.1f} | {x['speedup_vs_dense_cublas']:.2f} | "
                f"{x['spmm_graph_us']:.2f} | {x['dense_cublas_graph_us']:.2f} | {x['speedup_graph']:.2f} | "
                f"{x['useful_tflops']:.1f} | {fr} |")

    head = ("| workload | rows x k x ncols | N:M | kkeep | kernel (tile columns / accumulators / stack / blocks per stage) | "
            "SpMM us cold: median (min) | warm | dense cuBLAS us | x dense | graph replay us | dense cuBLAS graph us | x dense (graph) | "
            "useful TFLOP/s | roofline slot-aware / literal |\n|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for cfg, title in ((5, "Sweep (config 5) and 3:4"), (1, "Config 1"), (2, "Config 2"), (3, "Config 3: VGG-16 stand-in"),
                       (4, "Config 4: MobileNetV2 stand-in")):
        rows = [x for x in cells if x["config"] == cfg]
        if rows:
            o.append(f"\n**{title}** (`cells`)\n\n" + head + "\n" + "\n".join(row(x) for x in rows))
    if "summary" in d:
        o.append("\n**Per family** (`summary`; layers without a kept block left out; cold = each launch after an L2 flush in its own "
                 "event pair, graph = replay of 20 captured launches)\n\n| family | layers | ours us (cold) | dense cuBLAS us | x dense | "
                 "ours us (graph) | dense cuBLAS us (graph) | x dense (graph) | useful TFLOP/s | roofline min / median / max | "
                 "faster than dense cold / graph |\n|---|---|---|---|---|---|---|---|---|---|---|")
        for k, v in d["summary"].items():
            if "spmm_us_sum" in v:
                o.append(f"| {k} | {v['layers']} | {v['spmm_us_sum']:.1f} | {v['dense_cublas_us_sum']:.1f} | {v['speedup_vs_dense_cublas']:.2f} | "
                         f"{v['spmm_graph_us_sum']:.1f} | {v['dense_cublas_graph_us_sum']:.1f} | {v['speedup_graph']:.2f} | "
                         f"{v['useful_tflops']:.1f} | {v['roofline_frac_min']:.2f} / {v['roofline_frac_median']:.2f} / {v['roofline_frac_max']:.2f} | "
                         f"{v['faster_than_dense']} / {v['faster_than_dense_graph']} of {v['layers']} |")
        lo = d["summary"]["sweep_keep_le_0.5"]
        o.append(f"\nSweep cells with keep <= 0.5: {lo['at_or_above_60pct_of_roofline']} of {lo['cells']} at or above 0.60 of the "
                 f"slot-aware roofline, {lo['faster_than_dense']} of {lo['cells']} faster than dense cuBLAS.")
    for t in d.get("two_addend_form", []):
        o.append(f"`two_addend_form` {t['workload']}: dense tiles {t['dense']['spmm_us']:.1f} us, two 2:4 addends "
                 f"{t['sparse2']['spmm_us']:.1f} us ({t['two_addends_over_dense']:.2f}x), max |difference| {t['max_abs_difference']:.4f}.")
    for t in d.get("pruning_iteration", []):
        o.append(f"`pruning_iteration` {t['network']}: {t['layers']} layers, {t['weights']} weights, {t['samples']} gradient samples, "
                 f"{t['iteration_us']:.0f} us per iteration ({t['launches']} launches), oracle {t.get('oracle_us', 0) / 1e3:.0f} ms, "
                 f"kept counts equal: {t.get('matches_oracle')}.")
    for t in d.get("global_rank", []):
        o.append(f"`global_rank` {t['network']}: {t['global_rank_us']:.1f} us ({t['rank_positions']} rank positions), oracle "
                 f"{t.get('oracle_us', 0):.0f} us, equal: {t.get('matches_oracle')}.")
    for t in d.get("conv", []):
        o.append(f"`conv` {t['workload']} {t['activation']}: gather {t['conv_us']:.1f} us, lowered product {t['lowered_spmm_us']:.1f}, "
                 f"dense cuBLAS on the lowered matrix {t['dense_cublas_lowered_us']:.1f}; identical to lowered: {t['identical_to_lowered']}.")
    if "saliency" in d:
        t = d["saliency"]
        o.append(f"`saliency` {t['workload']}: {t['us']:.1f} us, {t['achieved_gbs']:.0f} GB/s = {t['roofline_frac']:.2f} of the HBM peak.")
    return "\n".join(o)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="sweep_2:4_keep0.5",
                    help="sweep_<n>:<m>_keep<r> (4096x4096x8192, block 128x64), config1, config2, or a layer name "
                         "of config 3 / 4 (vgg16_conv<i>, mbv2_b<i>_expand, mbv2_b<i>_project, mbv2_last)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cells", action="store_true", help="skip the per-layer / per-cell SpMM timings")
    ap.add_argument("--cell-iters", type=int, default=50, help="timed launches per cell and protocol")
    ap.add_argument("--render", metavar="JSON_FILE", help="print the markdown tables of a stored JSON line and exit")
    args = ap.parse_args()
    if args.render:
        print(render_markdown(json.loads([l for l in open(args.render) if l.startswith("{")][-1])))
        return
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    layer = pick_layer(args.workload)
    if args.impl == "reference":
        run_reference(args, layer, rank)
    else:
        run_ours(args, layer, rank, world)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the stacked-LSTM forward pass on B200.

Default run (one JSON line on stdout):
    python bench.py [--gpus N] [--steps K] [--warmup W]
A step is one lstm_forward over the large language-model workload (2 layers, 1500 -> 1500, T = 35,
batch 1, bf16 weights / fp32 state): input projection for all timesteps + serial recurrence, every
layer.  `value` is microseconds per sequence with inputs resident in device memory; `e2e` is the same
through lstm_forward_host with pinned host buffers (copies inside the timed region).  With N > 1 each
rank runs an independent replica (batch columns and sequences never interact): no collective on the
data path, N sequences per step.

Other modes:
    --impl reference     time the fp64 CPU oracle on the same workload (host cores only)
    --sweep              latency vs hidden size (H = 128..2048 step 8) with the LHP analysis
    --matmul-sweep       dense (tensor-core) vs sparse (CSR) matrix product at batch 16, d = 128..2048
    --workload NAME      cfg1 | cfg2 | cfg2_b20 | cfg4_10 | cfg4_05 | cfg4_10_csr | cfg4_05_csr |
                         cfg5 | cfg5_b16 (default cfg2)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import lstm_workloads as wl  # noqa: E402

FALLBACK_HBM_GBS = 6650.0


def pick_workload(name: str):
    table = {
        "cfg1": (wl.config1(), "dense"),
        "cfg2": (wl.config2(1), "dense"),
        "cfg2_b20": (wl.config2(20), "dense"),
        "cfg4_10": (wl.config4(0.10), "dense"),
        "cfg4_05": (wl.config4(0.05), "dense"),
        "cfg4_10_csr": (wl.config4(0.10), "csr"),
        "cfg4_05_csr": (wl.config4(0.05), "csr"),
        "cfg5": (wl.config5(1), "dense"),
        "cfg5_b16": (wl.config5(16), "dense"),
        # H-LSTM cell (one ReLU hidden layer of the cell's width inside each gate), the paper's own models:
        # one layer of width 1500 for the language model, three bidirectional layers of width 800 for speech
        "hlstm_ptb": (wl.config2(1).with_(name="hlstm_ptb_1x1500_B1", layers=1), "hlstm"),
        "hlstm_ds2": (wl.config5(1).with_(name="hlstm_ds2_3x2x800_B1", layers=3), "hlstm"),
    }
    return table[name]


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            d = json.loads(p.read_text())
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def measured_traffic(kernel: str, workload: str, source: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary
    profiles/<kernel>_<workload>.md, or None when there is none or the kernel's source has changed since
    the counters were taken (the summary records the sha256 of the source file it profiled)."""
    import hashlib
    import re
    f = ROOT / "profiles" / f"{kernel}_{workload}.md"
    src = ROOT / "paper_1901_10997_b200" / "csrc" / source
    if not (f.exists() and src.exists()):
        return None
    text = f.read_text()
    m_sha = re.search(r"source_sha256:\s*([0-9a-f]{64})", text)
    m_tr = re.search(r"traffic_bytes_per_launch:\s*([0-9]+)", text)
    if not (m_sha and m_tr) or hashlib.sha256(src.read_bytes()).hexdigest() != m_sha.group(1):
        return None
    return int(m_tr.group(1))


def make_inputs(w: wl.Workload, mode: str):
    return wl.make_hlstm(w, w.hidden) if mode == "hlstm" else wl.make(w)


def oracle_forward(w: wl.Workload, mode: str, weights, xs):
    import oracle
    if mode == "hlstm":
        return oracle.forward_hlstm(weights, xs, layers=w.layers, bidir=w.bidir, hidden=w.hidden, gate_hidden=w.hidden)
    return oracle.forward(weights, xs, layers=w.layers, bidir=w.bidir, hidden=w.hidden)


def recurrence_bytes_per_launch(w: wl.Workload, nnz_per_layer=None) -> float:
    """Algorithmic bytes one recurrent-kernel launch (one layer, all T steps, all directions) needs if
    nothing were resident: per step and direction the recurrent matrix once (4H*H*w bytes dense, or
    nnz*(value + 16-bit column) + row offsets for CSR), h read and written (B*H*8), and the
    projection row read (B*4H*4)."""
    H, B, T, D = w.hidden, w.B, w.T, w.dirs
    wbytes = 2 if w.dtype == "bf16" else 4
    if nnz_per_layer == "hlstm":
        mat = 2 * 4.0 * H * H * wbytes + B * 4.0 * H * 8.0      # Uh and W, plus the hidden-layer values exchanged
    elif nnz_per_layer is None:
        mat = 4.0 * H * H * wbytes
    else:
        mat = nnz_per_layer / D * (wbytes + 2) + (4 * H + 1) * 4
    return T * D * (mat + B * H * 8.0 + B * 4.0 * H * 4.0)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if r & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_time(w: wl.Workload, weights, x, target_seconds=12.0, max_reps=400, mode="dense"):
    """Times the oracle as it stands on a bounded sample: whole sequences of the workload (for B > 1
    only the first batch column), repeated until ~target_seconds of wall time have passed."""
    import oracle
    xs = x[:, :1] if w.B > 1 else x
    t0 = time.perf_counter()
    oracle_forward(w, mode, weights, xs)
    first = time.perf_counter() - t0
    reps = int(max(1, min(max_reps, target_seconds / max(first, 1e-6))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle_forward(w, mode, weights, xs)
    per_seq = (time.perf_counter() - t0) / reps
    return per_seq, reps, oracle.threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, _mode = pick_workload(args.workload)
    weights, x = make_inputs(w, _mode)
    import oracle
    xs = x[:, :1] if w.B > 1 else x
    for _ in range(min(args.warmup, 1)):
        oracle_forward(w, _mode, weights, xs)
    steps = max(1, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_forward(w, _mode, weights, xs)
    per_seq = (time.perf_counter() - t0) / steps
    us = per_seq * 1e6
    sample = f"{steps} whole sequences of {w.name} (T={w.T}, one batch column per step), fp64 oracle"
    print(json.dumps({
        "impl": "reference", "metric": "us_per_sequence", "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": per_seq * 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "layers": w.layers, "hidden": w.hidden, "T": w.T, "B": 1},
        "cpu_baseline": {"value": us, "unit": "us", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (the slowest replica sets the job's
    time); identity without a process group."""
    import torch
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(world: int, seqs_per_replica: int, ms_per_step: float):
    """Replicas only: every rank runs the same workload on its own sequences, so one step of the job
    processes world * B sequences in the slowest rank's step time.  Returns (sequences per step,
    microseconds per sequence, sequences per second)."""
    seqs = world * seqs_per_replica
    return seqs, ms_per_step * 1e3 / seqs, seqs / (ms_per_step * 1e-3)


def flush_l2(buf):
    buf.zero_()


def time_steps(fn, steps, warmup, flush_buf, torch):
    """Per-step CUDA-event timing on the current stream; L2 is flushed between steps outside the
    event pairs.  Returns the list of per-step milliseconds."""
    for _ in range(warmup):
        flush_l2(flush_buf)
        fn()
    torch.cuda.synchronize()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(steps):
        flush_l2(flush_buf)
        starts[i].record()
        fn()
        ends[i].record()
    torch.cuda.synchronize()
    return [s.elapsed_time(e) for s, e in zip(starts, ends)]


def run_gpu(args):
    import torch
    import paper_1901_10997_b200 as pkg

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w, mode = pick_workload(args.workload)
    weights, x = make_inputs(w, mode)

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        per_seq, reps, cores = oracle_time(w, weights, x, mode=mode)
        cpu = {"value": per_seq * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
               "sample": f"{reps} whole sequences of {w.name} (T={w.T}, one batch column each) after one warm-up"}

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod

    if mode == "hlstm":
        model = pkg.HLSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, gate_hidden=w.hidden, bidir=w.bidir,
                          dtype=w.dtype, max_T=w.T, max_B=w.B)
    else:
        model = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir, dtype=w.dtype,
                         exec_mode=mode, max_T=w.T, max_B=w.B)
    dev = torch.device("cuda", local_rank)
    xd = torch.from_numpy(x).to(dev)
    out = (torch.empty((w.T, w.B, w.dirs * w.hidden), device=dev),
           torch.empty((w.layers * w.dirs, w.B, w.hidden), device=dev),
           torch.empty((w.layers * w.dirs, w.B, w.hidden), device=dev))
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def step():
        model.forward(xd, out=out)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- timed region: device-resident inputs
    barrier()
    with ClockSampler(local_rank) as clocks:
        ms = time_steps(step, args.steps, max(args.warmup, 3), flush_buf, torch)
    barrier()
    model.check()
    total_ms = sum(ms)
    launches_per_fwd = model.info()["launches_per_forward"]

    # ---- same region again with the library's per-kernel events, for the roofline of the dominant kernel
    model.profile_enable(True)
    rec_ms, rec_n, proj_ms, stage_ms = 0.0, 0, 0.0, 0.0
    for i in range(args.steps + 3):
        flush_l2(flush_buf)
        step()
        n, t = model.profile_read()
        if i >= 3:
            rec_ms += t[pkg.LSTM_K_RECUR]; rec_n += n[pkg.LSTM_K_RECUR]
            proj_ms += t[pkg.LSTM_K_PROJ]; stage_ms += t[pkg.LSTM_K_STAGE]
    model.profile_enable(False)

    # ---- end to end through the host-buffer entry point (pinned buffers, copies inside the timing)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty((w.T, w.B, w.dirs * w.hidden)).pin_memory()
    hTh = torch.empty((w.layers * w.dirs, w.B, w.hidden)).pin_memory()
    cTh = torch.empty_like(hTh).pin_memory()
    st = torch.cuda.current_stream().cuda_stream
    for _ in range(3):
        model.forward_host(xh, y=yh, hT=hTh, cT=cTh, stream=st)
    barrier()
    e2e_steps = args.steps
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        flush_l2(flush_buf)
        model.forward_host(xh, y=yh, hT=hTh, cT=cTh, stream=st)
    torch.cuda.synchronize()
    e2e_total = time.perf_counter() - t0
    # the flush is outside the metric: time it separately and subtract
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        flush_l2(flush_buf)
    torch.cuda.synchronize()
    e2e_total -= time.perf_counter() - t0
    barrier()

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_total * 1e3], dist, dev)

    if rank == 0:
        ms_per_step = total_ms / args.steps
        seqs, us_per_seq, seqs_per_sec = job_throughput(world, w.B, ms_per_step)
        peak, peak_kind = measured_peaks()
        nnz = None
        if mode == "csr":
            nnz = float(np.mean([sum(int(np.count_nonzero(weights[l * w.dirs + d]["mask_h"])) for d in range(w.dirs))
                                 for l in range(w.layers)]))
        alg_bytes = recurrence_bytes_per_launch(w, "hlstm" if mode == "hlstm" else nnz)
        rec_avg_ms = rec_ms / max(rec_n, 1)
        achieved = alg_bytes / (rec_avg_ms * 1e-3) / 1e9 if rec_avg_ms > 0 else None
        info = model.info()
        kernel_name, kernel_src = (("hlstm_mma_kernel", "hlstm_mma.cu") if mode == "hlstm" else
                                   ("recur_tc_kernel", "recur_tc.cu") if info.get("recur_batched_tensor_core")
                                   else ("recur_mma_kernel", "recur_mma.cu") if info.get("recur_register_resident")
                                   else ("recur_kernel", "recur.cu"))
        traffic = measured_traffic(kernel_name, args.workload, kernel_src)
        line = {
            "metric": "us_per_sequence", "value": us_per_seq, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": ("bf16" if w.dtype == "bf16" else "f32"),
            "data": "synthetic",
            "config": {"workload": w.name, "layers": w.layers, "dirs": w.dirs, "in_dim": w.in_dim, "hidden": w.hidden,
                       "T": w.T, "B": w.B, "exec_mode": mode, "weights": w.dtype, "state": "fp32", "l2": "flushed between timed steps (256 MiB write)",
                       "parallelism": f"replicas x{world}"},
            "sequences_per_sec": seqs_per_sec,
            "step_ms_p10_p50_p90": [float(np.percentile(ms, q)) for q in (10, 50, 90)],
            "clocks": clocks.summary(),
            "gpu_launches": int(launches_per_fwd * args.steps),
            "e2e": {"value": e2e_ms * 1e3 / e2e_steps / seqs, "unit": "us",
                    "h2d_bytes_per_step": int(x.nbytes),
                    "d2h_bytes_per_step": int(yh.numel() * 4 + hTh.numel() * 4 + cTh.numel() * 4)},
            "roofline": {"bound": "hbm", "kernel": f"{kernel_name} (one launch = one layer, all T steps)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": (achieved / peak if achieved else None), "peak_kind": f"of {peak_kind}",
                         "traffic": traffic, "algorithmic_bytes_per_launch": alg_bytes,
                         "avg_launch_ms": rec_avg_ms,
                         "us_per_timestep": rec_avg_ms * 1e3 / w.T,
                         "note": "the recurrent matrix stays on-chip (registers / shared memory) for the whole "
                                 "sequence, so the fraction of the per-step HBM weight-read bound may exceed 1"},
            "kernel_ms_per_forward": {"stage": stage_ms / args.steps, "projection": proj_ms / args.steps,
                                      "recurrence": rec_ms / args.steps},
            "library": model.info(),
        }
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))
    model.close()
    if dist is not None:
        dist.destroy_process_group()


def lhp_analysis(hs, lat, eps):
    """Latency-hysteresis points of a measured curve (paper, Section 3) through the library's own
    helper: returns (sorted LHP sizes, redundancy in percent = (1 - #LHP / #points) * 100)."""
    import paper_1901_10997_b200 as pkg
    rc, flags, count = pkg.lstm_lhp_points(list(hs), list(lat), eps)
    if rc != pkg.LSTM_OK:
        raise RuntimeError(f"lstm_lhp_points failed with code {rc}")
    return sorted(h for h, f in zip(hs, flags) if f), (1 - count / len(hs)) * 100.0


def run_sweep(args):
    """Latency against hidden width with the hysteresis analysis (paper, Section 3).  Shape "cfg3": one
    layer, input = hidden = H, T = 35, batch 1 (the recurrent stack of Figure 2's kind).  Shape "ds2": the
    speech-model stack (5 bidirectional layers, 1312 -> H, then 2H -> H, T = 400) at batch 16, the
    setting of the paper's Figure 3."""
    import torch
    import paper_1901_10997_b200 as pkg
    dev = torch.device("cuda", 0)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    outdir = ROOT / "gpurun_out"
    outdir.mkdir(exist_ok=True)
    ds2 = args.sweep_shape == "ds2"
    default_sizes = list(range(256, 1536 + 1, 16)) if ds2 else wl.config3_sizes()
    sizes = default_sizes if not args.sweep_sizes else [int(s) for s in args.sweep_sizes.split(",")]
    parity_sizes = set(sizes) if not ds2 else {sizes[0], sizes[len(sizes) // 2], sizes[-1]}
    rows = []
    for H in sizes:
        w = wl.config5_width(H, 16) if ds2 else wl.config3(H)
        weights, x = wl.make(w)
        D = 2 if w.bidir else 1
        m = pkg.LSTM(weights, layers=w.layers, in_dim=w.in_dim, hidden=H, bidir=w.bidir, dtype="bf16", max_T=w.T, max_B=w.B)
        xd = torch.from_numpy(x).to(dev)
        out = (torch.empty((w.T, w.B, D * H), device=dev), torch.empty((w.layers * D, w.B, H), device=dev),
               torch.empty((w.layers * D, w.B, H), device=dev))
        ms = time_steps(lambda: m.forward(xd, out=out), args.steps, max(args.warmup, 3), flush_buf, torch)
        m.check()
        err = None
        if args.sweep_parity and H in parity_sizes:
            import oracle
            if ds2:
                # the oracle cannot walk 400 steps x 16 columns at every width: a 24-step call on the same
                # handle, all 16 columns on the GPU, the first column against the oracle
                Tp = 24
                got = m.forward(xd[:Tp].contiguous())
                m.check()
                ref = oracle.forward(weights, x[:Tp, :1], layers=w.layers, bidir=True, hidden=H)
                err = max(wl.rel_err(g[:, :1].cpu().numpy(), r)[0] for g, r in zip(got, ref))
            else:
                ref = oracle.forward(weights, x, layers=1, bidir=False, hidden=H)
                err = max(wl.rel_err(g.cpu().numpy(), r)[0] for g, r in zip(out, ref))
        info = m.info()
        m.close()
        rows.append({"H": H, "us_p50": float(np.percentile(ms, 50)) * 1e3, "us_p10": float(np.percentile(ms, 10)) * 1e3,
                     "us_p90": float(np.percentile(ms, 90)) * 1e3, "rows_streamed": info["rows_streamed"],
                     "threads": info["threads"], "batched_tensor_core": info.get("recur_batched_tensor_core"),
                     "max_rel_err": err})
        print(json.dumps(rows[-1]), file=sys.stderr, flush=True)
    hs = [r["H"] for r in rows]
    lat = [r["us_p50"] for r in rows]
    label = ("ds2 sweep: 5 bidirectional layers, 1312 -> H, T = 400, B = 16, bf16 weights; us per call (16 utterances)" if ds2
             else "cfg3 sweep: 1 layer, in = hidden = H, T = 35, B = 1, bf16 weights")
    res = {"workload": label, "steps": args.steps, "points": rows}
    for eps in (0.0, 0.005):
        lhps, red = lhp_analysis(hs, lat, eps)
        res[f"lhp_eps_{eps:g}"] = {"lhps": lhps, "count": len(lhps), "redundancy_percent": red}
    (outdir / ("sweep_ds2_b16.json" if ds2 else "sweep_cfg3.json")).write_text(json.dumps(res, indent=1))
    print(json.dumps({k: v for k, v in res.items() if k != "points"}))


def run_matmul_sweep(args):
    """The paper's Figures 1 and 2 on this GPU: one square matrix W [d x d] times a batch of 16 dense columns,
    dense (tensor-core projection, bf16 weights) against sparse (CSR projection over the surviving weights)
    at 90 % and 95 % sparsity, d = 128 .. 2048.  Timed with the library's per-kernel events (staging +
    projection kernels), L2 flushed between calls."""
    import torch
    import paper_1901_10997_b200 as pkg
    dev = torch.device("cuda", 0)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    outdir = ROOT / "gpurun_out"
    outdir.mkdir(exist_ok=True)
    rows = []
    for dsz in range(128, 2048 + 1, 64):
        H = dsz // 4
        row = {"d": dsz}
        for label, density, mode in (("dense_tc", 1.0, "dense"), ("csr_10", 0.10, "csr"), ("csr_05", 0.05, "csr")):
            w = wl.Workload(f"matmul_d{dsz}", 1, False, dsz, H, 16, 1, "bf16", 1.0 / np.sqrt(dsz), density=density,
                            seed=wl.SEED_BASE + dsz)
            weights, x = wl.make(w)
            m = pkg.LSTM(weights, layers=1, in_dim=dsz, hidden=H, dtype="bf16", exec_mode=mode, max_T=16, max_B=1)
            xd = torch.from_numpy(x).to(dev)
            out = torch.empty((16, 1, 1, 4 * H), device=dev)
            m.profile_enable(True)
            ts = []
            for i in range(args.steps + max(args.warmup, 3)):
                flush_l2(flush_buf)
                m.input_projection(xd, out=out)
                _n, t = m.profile_read()
                if i >= max(args.warmup, 3):
                    ts.append((t[pkg.LSTM_K_STAGE] + t[pkg.LSTM_K_PROJ]) * 1e3)
            m.check()
            if args.sweep_parity:
                import oracle
                ref = oracle.input_projection(weights, x, bidir=False, hidden=H)
                row[label + "_err"] = wl.rel_err(out.cpu().numpy().reshape(ref.shape), ref)[1]
            m.close()
            row[label + "_us"] = float(np.percentile(ts, 50))
        rows.append(row)
        print(json.dumps(row), file=sys.stderr, flush=True)
    (outdir / "matmul_sweep.json").write_text(json.dumps({"batch": 16, "steps": args.steps, "points": rows}, indent=1))
    wins = sum(1 for r in rows if r["csr_05_us"] < r["dense_tc_us"])
    print(json.dumps({"points": len(rows), "sparse_95_faster_than_dense_at": wins}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--matmul-sweep", action="store_true")
    ap.add_argument("--sweep-sizes", default="")
    ap.add_argument("--sweep-shape", default="cfg3", choices=["cfg3", "ds2"])
    ap.add_argument("--sweep-parity", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    elif args.matmul_sweep:
        run_matmul_sweep(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

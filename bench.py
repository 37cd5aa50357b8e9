#!/usr/bin/env python
"""Benchmark of the stacked-LSTM forward pass on B200.

Default run (one JSON line on stdout):
    python bench.py [--gpus N] [--steps K] [--warmup W]
A step is one lstm_forward over the large language-model workload (2 layers, 1500 -> 1500, T = 35,
batch 1, bf16 weights / fp32 state): input projection for all timesteps + serial recurrence, every
layer.  `value` is microseconds per sequence with inputs resident in device memory; `e2e` is the same
through lstm_forward_host with pinned host buffers (copies inside the timed region).  At one GPU the
line also carries short device-timed `legs` for the other workloads (batches of 20 and 16 sequences, the
pruned stack dense-with-zeros against CSR, the speech-shaped stack, the small fp32 stack), the on-chip
yardstick of the recurrent step (`roofline.on_chip`: the exchange-only step measured by the library's own
probe modes) and the fp64 CPU oracle timed on the host cores (all threads and one thread).
With N > 1 each rank runs an independent replica (batch columns and sequences never interact): no
collective on the data path, N sequences per step.  Started without a launcher, `--gpus N` starts the N
ranks itself (one process per GPU, rendezvous on 127.0.0.1).

Other modes:
    --impl reference     time the fp64 CPU oracle on the same workload (host cores only)
    --sweep              latency vs hidden size (H = 128..2048 step 8) with the LHP analysis
    --matmul-sweep       dense (tensor-core) vs sparse (CSR) matrix product at batch 16, d = 128..2048
    --wave-sweep         layer-wavefront kernel vs one launch per layer over H (2 layers, T = 35, batch 1)
    --workload NAME      cfg1 | cfg2 | cfg2_b20 | cfg4_10 | cfg4_05 | cfg4_10_csr | cfg4_05_csr |
                         cfg5 | cfg5_b16 | hlstm_ptb | hlstm_ds2 (default cfg2)
    --no-legs            headline workload only
    --out DIR            where the sweeps write their tables (default bench_out)
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import lstm_workloads as wl  # noqa: E402

FALLBACK_HBM_GBS = 6650.0

# legs of the default line at one GPU: (key, --workload name, timed steps)
LEGS = [("cfg2_b20", "cfg2_b20", 20), ("cfg5_b16", "cfg5_b16", 3), ("cfg5_b1", "cfg5", 5),
        ("cfg4_d10_dense_with_zeros", "cfg4_10", 20), ("cfg4_d10_csr", "cfg4_10_csr", 20),
        ("cfg4_d05_dense_with_zeros", "cfg4_05", 20), ("cfg4_d05_csr", "cfg4_05_csr", 20),
        ("cfg2_units_pruned_1197_compacted", "cfg2_rc", 20), ("cfg2_units_pruned_1197_zeros_kept", "cfg2_rc_zeros", 20),
        ("cfg2_units_pruned_1197_b20_compacted", "cfg2_rc_b20", 10), ("cfg2_units_pruned_1197_b20_zeros_kept", "cfg2_rc_b20_zeros", 10),
        ("cfg1_fp32_b20", "cfg1", 20)]


def pick_workload(name: str):
    table = {
        "cfg1": (wl.config1(), "dense"),
        "cfg2": (wl.config2(1), "dense"),
        "cfg2_b20": (wl.config2(20), "dense"),
        "cfg4_10": (wl.config4(0.10), "dense"),
        "cfg4_05": (wl.config4(0.05), "dense"),
        "cfg4_10_csr": (wl.config4(0.10), "csr"),
        "cfg4_05_csr": (wl.config4(0.05), "csr"),
        # row/column pruning (Section 4.2, Table 1 step (b)): 303 of 1500 hidden units per layer removed; run on the
        # surviving units (compacted) or with the zeros kept in the 1500-wide model
        "cfg2_rc": (wl.config2_units_pruned(1), "dense"),
        "cfg2_rc_zeros": (wl.config2_units_pruned(1), "dense"),
        "cfg2_rc_b20": (wl.config2_units_pruned(20), "dense"),
        "cfg2_rc_b20_zeros": (wl.config2_units_pruned(20), "dense"),
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
    """(DRAM bytes per launch, where they come from) of the dominant kernel from the committed ncu summary
    profiles/<kernel>_<workload>.md; (None, reason) when there is none or the kernel's source has changed
    since the counters were taken (the summary records the sha256 of the source file it profiled)."""
    import hashlib
    import re
    f = ROOT / "profiles" / f"{kernel}_{workload}.md"
    src = ROOT / "paper_1901_10997_b200" / "csrc" / source
    if not (f.exists() and src.exists()):
        return None, "no ncu summary for this kernel and workload"
    text = f.read_text()
    m_sha = re.search(r"source_sha256:\s*([0-9a-f]{64})", text)
    m_tr = re.search(r"traffic_bytes_per_launch:\s*([0-9]+)", text)
    if not (m_sha and m_tr):
        return None, f"profiles/{f.name} carries no counters"
    if hashlib.sha256(src.read_bytes()).hexdigest() != m_sha.group(1):
        return None, f"profiles/{f.name} was taken from an earlier revision of {source}"
    return int(m_tr.group(1)), f"profiles/{f.name} (one ncu capture, dram__bytes_read.sum + dram__bytes_write.sum; not measured in this run)"


def make_inputs(w: wl.Workload, mode: str):
    if mode == "hlstm":
        return wl.make_hlstm(w, w.hidden)
    weights, x = wl.make(w)
    if w.name.startswith("cfg2_units_pruned"):
        weights, _removed = wl.prune_units(w, weights, 1197)
    return weights, x


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
            self._stop.wait(0.005)

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


def oracle_time_one_thread(workload: str, reps: int = 3):
    """The same oracle on ONE host thread: a child process started with OMP_NUM_THREADS=1 (the thread count of
    an OpenMP library is fixed when it loads), whole sequences of the workload, one batch column.  Returns
    microseconds per sequence, or None if the child failed."""
    code = ("import sys, time, json; sys.path.insert(0, %r); import bench; "
            "w, mode = bench.pick_workload(%r); weights, x = bench.make_inputs(w, mode); xs = x[:, :1]; "
            "bench.oracle_forward(w, mode, weights, xs); t0 = time.perf_counter(); "
            "[bench.oracle_forward(w, mode, weights, xs) for _ in range(%d)]; "
            "import oracle; print(json.dumps({'us': (time.perf_counter() - t0) / %d * 1e6, 'threads': oracle.threads()}))"
            % (str(ROOT), workload, reps, reps))
    env = dict(os.environ, OMP_NUM_THREADS="1")
    try:
        r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
        d = json.loads(r.stdout.strip().splitlines()[-1])
        return float(d["us"]) if int(d["threads"]) == 1 else None
    except Exception:
        return None


def workload_config(w: wl.Workload, mode: str, world: int = 1):
    return {"workload": w.name, "layers": w.layers, "dirs": w.dirs, "in_dim": w.in_dim, "hidden": w.hidden,
            "T": w.T, "B": w.B, "exec_mode": mode, "weights": w.dtype, "state": "fp32",
            "l2": "flushed between timed steps (256 MiB write)", "parallelism": f"replicas x{world}"}


def run_reference(args):
    """The reference arm: the fp64 oracle as it stands on the host cores, same workload and metric.  A step is
    one whole sequence (one batch column) of the workload.  --steps / --warmup are honoured unless the run
    would pass three minutes, in which case fewer steps are timed and the line says how many."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, mode = pick_workload(args.workload)
    weights, x = make_inputs(w, mode)
    import oracle
    xs = x[:, :1] if w.B > 1 else x
    budget = 180.0
    t_begin = time.perf_counter()
    t0 = time.perf_counter()
    oracle_forward(w, mode, weights, xs)
    first = time.perf_counter() - t0
    warm = max(0, args.warmup - 1)
    warm = int(min(warm, max(0, (0.25 * budget - first) / max(first, 1e-9))))
    for _ in range(warm):
        oracle_forward(w, mode, weights, xs)
    left = budget - (time.perf_counter() - t_begin)
    steps = int(max(1, min(args.steps, left / max(first, 1e-9))))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_forward(w, mode, weights, xs)
    per_seq = (time.perf_counter() - t0) / steps
    us = per_seq * 1e6
    sample = f"{steps} whole sequences of {w.name} (T={w.T}, one batch column per step), fp64 oracle"
    cfg = workload_config(w, mode, 1)
    cfg["l2"] = "not applicable (host)"
    cfg["parallelism"] = "host threads (OpenMP over independent outputs)"
    print(json.dumps({
        "impl": "reference", "metric": "us_per_sequence", "value": us, "unit": "us", "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, warm + 1), "ms_per_step": per_seq * 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": cfg,
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


def time_back_to_back(fn, calls, reps, torch):
    """`calls` calls inside ONE event pair, `reps` pairs: the per-call time no longer depends on the tick of the
    event clock; L2 stays warm (the serving-loop case).  Returns the median per-call milliseconds."""
    fn()
    torch.cuda.synchronize()
    out = []
    for _ in range(reps):
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(calls):
            fn()
        e.record()
        torch.cuda.synchronize()
        out.append(s.elapsed_time(e) / calls)
    return float(np.median(out))


def trimmed_mean(ms, drop=0.1):
    """Mean without the slowest `drop` share of the samples: unlike a median it resolves differences below the
    tick of the event clock (the ticks average out over the samples)."""
    v = sorted(ms)
    keep = v[:max(1, int(round(len(v) * (1.0 - drop))))]
    return float(sum(keep) / len(keep))


def kernel_of(info, mode):
    if mode == "hlstm":
        return "hlstm_mma_kernel", "hlstm_mma.cu"
    if mode == "csr":
        return ("recur_csr_kernel", "recur_csr.cu") if info.get("recur_csr_register_resident") else ("recur_kernel", "recur.cu")
    if info.get("recur_batched_tensor_core"):
        return "recur_tc_kernel", "recur_tc.cu"
    if info.get("recur_register_resident"):
        return "recur_mma_kernel", "recur_mma.cu"
    return "recur_kernel", "recur.cu"


class GpuCase:
    """One workload on one device: handle, device buffers, and the timed regions."""

    def __init__(self, torch, pkg, workload_name, dev, flush_buf, weights_cache=None):
        self.torch, self.pkg = torch, pkg
        self.name = workload_name
        self.w, self.mode = pick_workload(workload_name)
        w = self.w
        key = (w.seed, w.layers, w.bidir, w.in_dim, w.hidden, w.dtype, w.density, self.mode == "hlstm")
        if weights_cache is not None and key in weights_cache and weights_cache[key][1].shape[1] >= w.B:
            self.weights, xs = weights_cache[key]
            self.x = np.ascontiguousarray(xs[:, :w.B])
        else:
            self.weights, self.x = make_inputs(w, self.mode)
            if weights_cache is not None:
                weights_cache[key] = (self.weights, self.x)
        if self.mode == "hlstm":
            self.model = pkg.HLSTM(self.weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, gate_hidden=w.hidden,
                                   bidir=w.bidir, dtype=w.dtype, max_T=w.T, max_B=w.B)
        else:
            keep_zeros = workload_name.endswith("_zeros")
            force = workload_name.startswith("cfg2_rc")
            old = os.environ.get("LSTM_B200_COMPACT")
            if force:
                os.environ["LSTM_B200_COMPACT"] = "0" if keep_zeros else "1"
            try:
                self.model = pkg.LSTM(self.weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir,
                                      dtype=w.dtype, exec_mode=self.mode, max_T=w.T, max_B=w.B)
            finally:
                if force:
                    if old is None:
                        os.environ.pop("LSTM_B200_COMPACT", None)
                    else:
                        os.environ["LSTM_B200_COMPACT"] = old
        self.dev = dev
        self.flush_buf = flush_buf
        self.xd = torch.from_numpy(self.x).to(dev)
        self.out = (torch.empty((w.T, w.B, w.dirs * w.hidden), device=dev),
                    torch.empty((w.layers * w.dirs, w.B, w.hidden), device=dev),
                    torch.empty((w.layers * w.dirs, w.B, w.hidden), device=dev))

    def step(self):
        self.model.forward(self.xd, out=self.out)

    def timed(self, steps, warmup):
        ms = time_steps(self.step, steps, warmup, self.flush_buf, self.torch)
        self.model.check()
        return ms

    def kernel_split(self, steps, warmup=3):
        """The same region again with the library's per-kernel events: (recurrence ms, recurrence launches,
        projection ms, staging ms), totals over `steps` forwards."""
        pkg, m = self.pkg, self.model
        m.profile_enable(True)
        rec_ms, rec_n, proj_ms, stage_ms = 0.0, 0, 0.0, 0.0
        for i in range(steps + warmup):
            flush_l2(self.flush_buf)
            self.step()
            n, t = m.profile_read()
            if i >= warmup:
                rec_ms += t[pkg.LSTM_K_RECUR]; rec_n += n[pkg.LSTM_K_RECUR]
                proj_ms += t[pkg.LSTM_K_PROJ]; stage_ms += t[pkg.LSTM_K_STAGE]
        m.profile_enable(False)
        return rec_ms, rec_n, proj_ms, stage_ms

    def nnz(self):
        if self.mode != "csr":
            return None
        w = self.w
        return float(np.mean([sum(int(np.count_nonzero(self.weights[l * w.dirs + d]["mask_h"])) for d in range(w.dirs))
                              for l in range(w.layers)]))

    def roofline(self, rec_ms, rec_n, peak, peak_kind, fused=False):
        w = self.w
        alg_bytes = recurrence_bytes_per_launch(w, "hlstm" if self.mode == "hlstm" else self.nnz())
        if fused:
            # the launch also computes its layer's input projection: the input matrix and the activations once
            wbytes = 2 if w.dtype == "bf16" else 4
            in_avg = (w.in_dim + (w.layers - 1) * w.dirs * w.hidden) / w.layers
            alg_bytes += w.dirs * 4.0 * w.hidden * in_avg * wbytes + w.T * w.B * in_avg * 4.0
        rec_avg_ms = rec_ms / max(rec_n, 1)
        achieved = alg_bytes / (rec_avg_ms * 1e-3) / 1e9 if rec_avg_ms > 0 else None
        info = self.model.info()
        kernel_name, kernel_src = kernel_of(info, self.mode)
        traffic, source = measured_traffic(kernel_name, self.name, kernel_src)
        steps_per_launch = w.T * (2 if (w.dirs == 2 and info.get("ctas_per_dir") == info.get("sm_count")) else 1)
        return {"bound": "hbm", "kernel": f"{kernel_name} (one launch = one layer, all T steps" + (", its input projection in the prologue)" if fused else ")"),
                "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": (achieved / peak if achieved else None), "peak_kind": f"of {peak_kind}",
                "traffic": traffic, "traffic_source": source, "algorithmic_bytes_per_launch": alg_bytes,
                "avg_launch_ms": rec_avg_ms, "us_per_timestep": rec_avg_ms * 1e3 / steps_per_launch,
                "note": "the recurrent matrix stays on-chip (registers / shared memory) for the whole sequence, so the "
                        "fraction of the per-step HBM weight-read bound may exceed 1; on_chip holds the bound that binds"}

    def on_chip(self, steps):
        """The yardstick that binds once the matrix is on-chip: the dependency chain of one step.  Uses the
        library's probe modes (parts of the step left out) on this very handle and workload; every figure is the
        recurrent kernel's launch time / T, prologue included, all from the measurement build of the kernel (projection as a
        launch of its own, so that every mode has the same prologue)."""
        pkg, m, w = self.pkg, self.model, self.w
        try:
            m.probe(0)
        except pkg.LstmError:
            return None
        res = {}
        modes = [("step_us_probe_build", pkg.LSTM_PROBE_WHOLE_STEP),
                 ("empty_step_us", pkg.LSTM_PROBE_NO_PRODUCTS | pkg.LSTM_PROBE_NO_GATES),
                 ("exchange_and_gates_us", pkg.LSTM_PROBE_NO_PRODUCTS),
                 ("compute_only_us", pkg.LSTM_PROBE_NO_EXCHANGE),
                 ("products_only_us", pkg.LSTM_PROBE_NO_EXCHANGE | pkg.LSTM_PROBE_NO_GATES)]
        try:
            for key, mask in modes:
                m.probe(mask)
                rec_ms, rec_n, _p, _s = self.kernel_split(steps)
                m.check()
                res[key] = rec_ms / max(rec_n, 1) * 1e3 / w.T
        finally:
            m.probe(0)
        self.step()                 # leave valid outputs behind
        m.check()
        # The production step, from the production instantiation of the same kernel with the projection as a launch
        # of its own (same prologue as the probe modes): a second handle on the same weights with the fused prologue
        # switched off.  The probe builds carry run-time tests in the step (about 12 % on the whole step), so
        # step_us_probe_build is above step_us; the modes that leave parts out are what they are for.
        old = os.environ.get("LSTM_B200_FUSE")
        os.environ["LSTM_B200_FUSE"] = "0"
        try:
            plain = pkg.LSTM(self.weights, layers=w.layers, in_dim=w.in_dim, hidden=w.hidden, bidir=w.bidir, dtype=w.dtype,
                             exec_mode=self.mode, max_T=w.T, max_B=w.B)
        finally:
            if old is None:
                os.environ.pop("LSTM_B200_FUSE", None)
            else:
                os.environ["LSTM_B200_FUSE"] = old
        keep = self.model
        self.model = plain
        try:
            rec_ms, rec_n, _p, _s = self.kernel_split(steps)
            plain.check()
        finally:
            self.model = keep
            plain.close()
        res["step_us"] = rec_ms / max(rec_n, 1) * 1e3 / w.T
        res["step_over_empty_step"] = res["step_us"] / res["empty_step_us"] if res.get("empty_step_us") else None
        res["what"] = ("per timestep = recurrent launch / T, prologue included; step_us: the production kernel with the projection as its own "
                       "launch; the rest measured by the library's probe builds (lstm_probe): empty_step = publish -> L2 -> poll + CTA barrier, "
                       "no products, no gate functions; compute_only = products + barrier + reduction + gates + stores without "
                       "waiting for other CTAs; the weights are read from the register file, so no shared-memory or HBM "
                       "bandwidth bounds the step: the exchange latency does")
        return res

    def close(self):
        self.model.close()


def run_gpu(args):
    import torch
    import paper_1901_10997_b200 as pkg

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w, mode = pick_workload(args.workload)
    cache = {}
    weights, x = make_inputs(w, mode)
    cache[(w.seed, w.layers, w.bidir, w.in_dim, w.hidden, w.dtype, w.density, mode == "hlstm")] = (weights, x)

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        # before the first CUDA call: the one-thread sample runs in a child process
        one_thread_us = oracle_time_one_thread(args.workload)
        per_seq, reps, cores = oracle_time(w, weights, x, mode=mode)
        cpu = {"value": per_seq * 1e6, "unit": "us", "cores": cores, "kind": "oracle",
               "sample": f"{reps} whole sequences of {w.name} (T={w.T}, one batch column each) after one warm-up",
               "value_1thread": one_thread_us,
               "sample_1thread": "3 whole sequences in a child process with OMP_NUM_THREADS=1"}

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod

    dev = torch.device("cuda", local_rank)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    case = GpuCase(torch, pkg, args.workload, dev, flush_buf, cache)
    model = case.model

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- timed region: device-resident inputs
    warmup = max(args.warmup, 3)
    barrier()
    with ClockSampler(local_rank) as clocks:
        ms = case.timed(args.steps, warmup)
        barrier()
        # the same region once more with the library's per-kernel events (the clocks are sampled over both)
        rec_ms, rec_n, proj_ms, stage_ms = case.kernel_split(args.steps)
    total_ms = sum(ms)
    launches_per_fwd = model.info()["launches_per_forward"]

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
        roof = case.roofline(rec_ms, rec_n, peak, peak_kind, fused=(proj_ms == 0.0 and stage_ms == 0.0))
        gpu_launches = int(launches_per_fwd * args.steps)
        if world == 1 and not args.no_legs:
            oc = case.on_chip(min(args.steps, 20))
            if oc is not None:
                roof["on_chip"] = oc
        line = {
            "metric": "us_per_sequence", "value": us_per_seq, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": ("bf16" if w.dtype == "bf16" else "f32"),
            "data": "synthetic",
            "config": workload_config(w, mode, world),
            "sequences_per_sec": seqs_per_sec,
            "step_ms_p10_p50_p90": [float(np.percentile(ms, q)) for q in (10, 50, 90)],
            "clocks": clocks.summary(),
            "gpu_launches": gpu_launches,
            "e2e": {"value": e2e_ms * 1e3 / e2e_steps / seqs, "unit": "us",
                    "h2d_bytes_per_step": int(x.nbytes),
                    "d2h_bytes_per_step": int(yh.numel() * 4 + hTh.numel() * 4 + cTh.numel() * 4)},
            "roofline": roof,
            "kernel_ms_per_forward": {"stage": stage_ms / args.steps, "projection": proj_ms / args.steps,
                                      "recurrence": rec_ms / args.steps},
            "library": model.info(),
        }
        if cpu is not None:
            line["cpu_baseline"] = cpu
        case.close()
        if world == 1 and not args.no_legs and args.workload == "cfg2":
            line["legs"] = run_legs(torch, pkg, dev, flush_buf, cache, peak, peak_kind)
        print(json.dumps(line))
    else:
        case.close()
    if dist is not None:
        dist.destroy_process_group()


def run_legs(torch, pkg, dev, flush_buf, cache, peak, peak_kind):
    """The other workloads of the metric, each device-timed like the headline (L2 flushed between steps, CUDA
    events, 3 warm-up steps) with its own step count, so that the whole line stays within a minute or so."""
    legs = {}
    for key, name, steps in LEGS:
        t0 = time.perf_counter()
        try:
            case = GpuCase(torch, pkg, name, dev, flush_buf, cache)
        except Exception as e:      # a leg must not take the headline down with it
            legs[key] = {"error": str(e)}
            continue
        try:
            w = case.w
            with ClockSampler(dev.index or 0) as clocks:
                ms = case.timed(steps, 3)
            rec_ms, rec_n, proj_ms, stage_ms = case.kernel_split(min(steps, 5))
            nk = min(steps, 5)
            p50 = float(np.percentile(ms, 50))
            legs[key] = {
                "config": workload_config(w, case.mode),
                "steps": steps, "warmup": 3,
                "step_ms_p10_p50_p90": [float(np.percentile(ms, q)) for q in (10, 50, 90)],
                "ms_per_call": float(np.mean(ms)),
                "us_per_sequence": float(np.mean(ms)) * 1e3 / w.B,
                "sequences_per_sec": w.B / (float(np.mean(ms)) * 1e-3),
                "sequences_per_sec_p50": w.B / (p50 * 1e-3),
                "gpu_launches": int(case.model.info()["launches_per_forward"] * steps),
                "kernel_ms_per_forward": {"stage": stage_ms / nk, "projection": proj_ms / nk, "recurrence": rec_ms / nk},
                "roofline": case.roofline(rec_ms, rec_n, peak, peak_kind, fused=(proj_ms == 0.0 and stage_ms == 0.0 and case.mode == "dense" and w.dtype == "bf16")),
                "library": case.model.info(),
                "clocks": clocks.summary(),
                "wall_s": None,
            }
        except Exception as e:
            legs[key] = {"error": str(e)}
        finally:
            case.close()
        if isinstance(legs[key], dict) and "wall_s" in legs[key]:
            legs[key]["wall_s"] = round(time.perf_counter() - t0, 2)
    return legs


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
    setting of the paper's Figure 3.  Two timings per size: `us_cold` (one call per event pair, L2 flushed before
    it, mean without the slowest tenth, which resolves below the event clock's tick) and `us_warm` (enough calls
    back to back inside one event pair to span at least 200 us, L2 warm: the serving-loop case)."""
    import torch
    import paper_1901_10997_b200 as pkg
    dev = torch.device("cuda", 0)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    outdir = Path(args.out)
    outdir.mkdir(parents=True, exist_ok=True)
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
        fn = lambda: m.forward(xd, out=out)
        ms = time_steps(fn, args.steps, max(args.warmup, 3), flush_buf, torch)
        m.check()
        cold = trimmed_mean(ms)
        calls = max(1, int(np.ceil(0.2 / max(cold, 1e-4))))
        warm = time_back_to_back(fn, calls, 9 if not ds2 else 3, torch)
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
        rows.append({"H": H, "us_cold": cold * 1e3, "us_warm": warm * 1e3, "calls_per_event_pair": calls,
                     "us_p50": float(np.percentile(ms, 50)) * 1e3, "us_p10": float(np.percentile(ms, 10)) * 1e3,
                     "us_p90": float(np.percentile(ms, 90)) * 1e3, "rows_streamed": info["rows_streamed"],
                     "threads": info["threads"], "batched_tensor_core": info.get("recur_batched_tensor_core"),
                     "max_rel_err": err})
        print(json.dumps(rows[-1]), file=sys.stderr, flush=True)
    hs = [r["H"] for r in rows]
    label = ("ds2 sweep: 5 bidirectional layers, 1312 -> H, T = 400, B = 16, bf16 weights; us per call (16 utterances)" if ds2
             else "cfg3 sweep: 1 layer, in = hidden = H, T = 35, B = 1, bf16 weights")
    res = {"workload": label, "steps": args.steps, "points": rows}
    for which in ("us_warm", "us_cold"):
        lat = [r[which] for r in rows]
        for eps in (0.0, 0.005):
            lhps, red = lhp_analysis(hs, lat, eps)
            res[f"lhp_{which}_eps_{eps:g}"] = {"lhps": lhps, "count": len(lhps), "redundancy_percent": red}
    (outdir / ("sweep_ds2_b16.json" if ds2 else "sweep_cfg3.json")).write_text(json.dumps(res, indent=1))
    print(json.dumps({k: v for k, v in res.items() if k != "points"}))


def run_matmul_sweep(args):
    """The paper's Figures 1 and 2 on this GPU: one square matrix W [d x d] times a batch of 16 dense columns,
    dense (tensor-core projection, bf16 weights) against sparse (CSR projection over the surviving weights)
    at 90 % and 95 % sparsity, d = 128 .. 2048.  Every variant is timed the same way: the whole
    lstm_input_projection call (staging where the variant has it, product, re-layout of the result), enough
    calls back to back inside one event pair to span 200 us (`_us`, L2 warm) and, beside it, one call per event
    pair with L2 flushed (`_cold_us`, mean without the slowest tenth)."""
    import torch
    import paper_1901_10997_b200 as pkg
    dev = torch.device("cuda", 0)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    outdir = Path(args.out)
    outdir.mkdir(parents=True, exist_ok=True)
    rows = []
    for dsz in range(128, 2048 + 1, 64):
        H = dsz // 4
        row = {"d": dsz}
        for label, density, mode in (("dense_tc", 1.0, "dense"), ("csr_10", 0.10, "csr"), ("csr_05", 0.05, "csr")):
            w = wl.Workload(f"matmul_d{dsz}", 1, False, dsz, H, 16, 1, "bf16", 1.0 / np.sqrt(dsz), density=density,
                            seed=wl.SEED_BASE + dsz)
            weights, x = wl.make(w)
            # the sparse arms walk the lists (by default a bf16 CSR handle would project on the tensor cores over a
            # dense copy of the matrix, which is the dense arm again)
            old_env = os.environ.get("LSTM_B200_PROJ")
            if mode == "csr":
                os.environ["LSTM_B200_PROJ"] = "csr"
            try:
                m = pkg.LSTM(weights, layers=1, in_dim=dsz, hidden=H, dtype="bf16", exec_mode=mode, max_T=16, max_B=1)
            finally:
                if old_env is None:
                    os.environ.pop("LSTM_B200_PROJ", None)
                else:
                    os.environ["LSTM_B200_PROJ"] = old_env
            xd = torch.from_numpy(x).to(dev)
            out = torch.empty((16, 1, 1, 4 * H), device=dev)
            fn = lambda: m.input_projection(xd, out=out)
            ms = time_steps(fn, args.steps, max(args.warmup, 3), flush_buf, torch)
            cold = trimmed_mean(ms)
            calls = max(1, int(np.ceil(0.2 / max(cold, 1e-4))))
            warm = time_back_to_back(fn, calls, 9, torch)
            m.check()
            if args.sweep_parity:
                import oracle
                ref = oracle.input_projection(weights, x, bidir=False, hidden=H)
                row[label + "_err"] = wl.rel_err(out.cpu().numpy().reshape(ref.shape), ref)[1]
            m.close()
            row[label + "_us"] = warm * 1e3
            row[label + "_cold_us"] = cold * 1e3
        rows.append(row)
        print(json.dumps(row), file=sys.stderr, flush=True)
    (outdir / "matmul_sweep.json").write_text(json.dumps({"batch": 16, "steps": args.steps, "points": rows}, indent=1))
    summary = {"points": len(rows)}
    for which in ("_us", "_cold_us"):
        summary["sparse_95_faster_than_dense" + which] = sum(1 for r in rows if r["csr_05" + which] < r["dense_tc" + which])
        summary["sparse_90_faster_than_dense" + which] = sum(1 for r in rows if r["csr_10" + which] < r["dense_tc" + which])
    print(json.dumps(summary))


def run_wave_sweep(args):
    """Layer-wavefront kernel against one launch per layer on the two-layer language-model shape (input = hidden
    = H, T = 35, batch 1, bf16 weights): microseconds per sequence for both, the same handle settings otherwise.
    Timed like the hidden-size sweep (`us_cold`: L2 flushed, one call per event pair; `us_warm`: calls back to
    back inside one pair)."""
    import torch
    import paper_1901_10997_b200 as pkg
    dev = torch.device("cuda", 0)
    flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    outdir = Path(args.out)
    outdir.mkdir(parents=True, exist_ok=True)
    sizes = [int(s) for s in args.sweep_sizes.split(",")] if args.sweep_sizes else [128, 200, 256, 384, 512, 640, 768, 896, 1000, 1024]
    layers = args.wave_layers
    rows = []
    for H in sizes:
        w = wl.Workload(f"wave_sweep_L{layers}_H{H}", layers, False, H, H, 35, args.wave_batch, "bf16", 1.0 / np.sqrt(H), seed=wl.SEED_BASE + 7 * H + layers)
        weights, x = wl.make(w)
        xd = torch.from_numpy(x).to(dev)
        out = (torch.empty((w.T, w.B, H), device=dev), torch.empty((layers, w.B, H), device=dev), torch.empty((layers, w.B, H), device=dev))
        row = {"H": H, "layers": layers, "B": w.B}
        old = os.environ.get("LSTM_B200_WAVE")
        try:
            for label, env in (("wavefront", "1"), ("per_layer", "0")):
                os.environ["LSTM_B200_WAVE"] = env
                m = pkg.LSTM(weights, layers=layers, in_dim=H, hidden=H, dtype="bf16", max_T=w.T, max_B=w.B)
                info = m.info()
                if label == "wavefront" and not info["layer_wavefront"]:
                    m.close()
                    row["wavefront_served"] = False
                    continue
                fn = lambda: m.forward(xd, out=out)
                ms = time_steps(fn, args.steps, max(args.warmup, 3), flush_buf, torch)
                m.check()
                cold = trimmed_mean(ms)
                warm = time_back_to_back(fn, max(1, int(np.ceil(0.2 / max(cold, 1e-4)))), 9, torch)
                m.check()
                row[label + "_us_cold"] = cold * 1e3
                row[label + "_us_warm"] = warm * 1e3
                row[label + "_launches"] = m.info()["launches_per_forward"]
                if args.sweep_parity:
                    import oracle
                    ref = oracle.forward(weights, x, layers=layers, bidir=False, hidden=H)
                    row[label + "_err"] = max(wl.rel_err(g.cpu().numpy(), r)[1] for g, r in zip(out, ref))
                m.close()
        finally:
            if old is None:
                os.environ.pop("LSTM_B200_WAVE", None)
            else:
                os.environ["LSTM_B200_WAVE"] = old
        rows.append(row)
        print(json.dumps(row), file=sys.stderr, flush=True)
    (outdir / f"wave_sweep_L{layers}_B{args.wave_batch}.json").write_text(json.dumps({"steps": args.steps, "points": rows}, indent=1))
    print(json.dumps({"points": len(rows),
                      "wavefront_faster_cold": [r["H"] for r in rows if r.get("wavefront_us_cold", 1e9) < r.get("per_layer_us_cold", 0)],
                      "wavefront_faster_warm": [r["H"] for r in rows if r.get("wavefront_us_warm", 1e9) < r.get("per_layer_us_warm", 0)]}))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_replicas(args):
    """`--gpus N` without a launcher: start the N ranks (one process per GPU) under torch's own launcher on
    127.0.0.1 and hand back its exit code; rank 0 prints the job's single JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(Path(__file__).resolve()), *sys.argv[1:]]
    return subprocess.call(cmd)


def run_replica_check(args):
    """The rank bookkeeping of the N-replica run with no GPU work (gloo): every rank joins the group, takes part
    in the barrier and the max-over-ranks reduction of a made-up step time (10 + rank ms), rank 0 prints."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    d = None
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
        d = dist
    total_ms, = max_over_ranks([10.0 + rank], d, torch.device("cpu"))
    seqs, us_per_seq, per_sec = job_throughput(world, 1, total_ms)
    if rank == 0:
        print(json.dumps({"replica_check": True, "n_gpus": world, "ms_per_step": total_ms, "sequences_per_step": seqs,
                          "value": us_per_seq, "sequences_per_sec": per_sec}))
    if d is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--matmul-sweep", action="store_true")
    ap.add_argument("--wave-sweep", action="store_true")
    ap.add_argument("--wave-layers", type=int, default=2)
    ap.add_argument("--wave-batch", type=int, default=1)
    ap.add_argument("--sweep-sizes", default="")
    ap.add_argument("--sweep-shape", default="cfg3", choices=["cfg3", "ds2"])
    ap.add_argument("--sweep-parity", action="store_true")
    ap.add_argument("--out", default=str(ROOT / "bench_out"))
    ap.add_argument("--replica-check", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.sweep or args.matmul_sweep or args.wave_sweep):
        raise SystemExit(spawn_replicas(args))
    if args.replica_check:
        run_replica_check(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    elif args.matmul_sweep:
        run_matmul_sweep(args)
    elif args.wave_sweep:
        run_wave_sweep(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

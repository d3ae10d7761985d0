#!/usr/bin/env python
"""Throughput of the LoRA projection layer (forward + backward) on B200.

A step is one pass of the whole hot path - forward (X A^T pass + GEMM with the rank-r product as an extra k-block, or the
fused kernel), then backward (dY B and X A^T in one skinny launch, the dX GEMM, dA and dB in one skinny launch) - for every
projection of the workload, over one batch of seeded synthetic input.  The default workload is the whole Llama-3-8B decoder
layer: seven projections (q, k, v, o, gate, up, down), T = 32768 packed tokens, r = 16, s = 2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload {0..5}] [--impl reference] [--quick]

Prints ONE JSON line: the headline workload's timed region (`value`), the same step looped for >= 2 s (`sustained`), per-stage
durations with their roofline fractions (`kernels`, `roofline`, `roofline_hbm`), the other workloads from short runs in the
same process (`per_config`), variants, the end-to-end figure with host buffers, and the CPU oracle timed beside it.
With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica on its own batch: the layer has no collective,
so the job's value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

L2_BYTES = 126 * 1024 * 1024
E2E_STREAMS = int(os.environ.get("LORA_BENCH_E2E_STREAMS", "8"))      # streams the projections of one end-to-end step rotate over (3: 136 ms, 4: 122 ms, 7: 116 ms per layer step)
SETTLE_S = 1.5                        # seconds of untimed steps before the timed region (on top of the W warm-up steps)
NF4_BAND_BYTES = 16 * 1024 * 1024      # scratch buffer of the banded Q+LoRA variant (the largest weight of the layer is 112 MiB)
METRIC = "lora_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu captures summarised under profiles/;
# an entry is valid only for the kernel source it was taken on (source_sha of the GEMM files, of the streaming kernel's) and
# for the stage and projection shape its key names.  Both captures ran on a smaller token count (the GEMM's at T = 16384, the
# streaming launches' at T = 8192) and are scaled by the tokens: GEMM traffic is per band of m-tiles and the number of bands
# grows with T; a streaming launch's traffic is the two streamed matrices, proportional to T.
NCU_TRAFFIC = {
    "gemm_sha": "528a6efb94fd7e1e",
    "gemm_bytes_per_launch": {"32768x14336x4096": 3798919680},       # 2 x (1444.2 + 455.3 MB) captured at T = 16384
    "stream_sha": "310b01e3e28131ab",
    "stream_bytes_per_launch": {                                      # 4 x the launches captured at T = 8192
        "sides:32768x4096x4096": 552556544, "grads:32768x4096x4096": 551930880,
        "sides:32768x4096x1024": 346225664, "grads:32768x4096x1024": 347225088,
        "sides:32768x4096x14336": 1235765248, "grads:32768x4096x14336": 1223817216,
        "sides:32768x14336x4096": 1241160704, "grads:32768x14336x4096": 1224769536}}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def source_sha(prefix: str) -> str:
    """sha of the kernel sources whose names start with `prefix` plus the shared headers (keys the stored ncu traffic)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2503_22673_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.startswith(prefix) or name in ("sm100_ptx.cuh", "kernels.h"):
            with open(os.path.join(csrc, name), "rb") as f:
                h.update(f.read())
    return h.hexdigest()[:16]


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi (every 20 ms, timestamped) while the GPU works."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        import tempfile
        self.proc = None
        self.out = tempfile.TemporaryFile(mode="w+")      # a file, not a pipe: a full pipe would stall nvidia-smi
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=self.out, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    @staticmethod
    def _epoch(stamp: str):
        import datetime
        try:
            return datetime.datetime.strptime(stamp.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, t0: float = None, t1: float = None):
        """Summary of the samples taken between host times t0 and t1 (all samples when none fall inside)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            self.proc.wait()
        self.out.seek(0)
        out = self.out.read()
        self.out.close()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = []
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                rows.append((self._epoch(parts[0]), float(parts[1]), float(parts[2]),
                             [n for n, v in zip(names, parts[3:7]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        self.rows = rows
        return self.window(t0, t1)

    def window(self, t0: float = None, t1: float = None, label: str = "timed region"):
        rows = getattr(self, "rows", [])
        inside = [r for r in rows if t0 is not None and r[0] is not None and t0 <= r[0] <= t1]
        window = label if inside else f"whole run (no sample fell inside the {label})"
        use = inside if inside else rows
        sm = [r[1] for r in use]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(r[2] for r in use) if use else None,
                "samples": len(use), "window": window, "reasons": sorted({n for r in use for n in r[3]})}


def max_over_ranks(value: float, device, world: int) -> float:
    """Slowest rank's figure (all ranks must call it); identity for a single process."""
    if world == 1:
        return float(value)
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, flops_per_rank_step: float, ms_step: float) -> float:
    """Whole-job TFLOP/s: every rank does one step's FLOPs in the slowest rank's time (replicas, weak scaling)."""
    return world * flops_per_rank_step / ms_step / 1e9


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def workload_name(idx: int) -> str:
    return {0: "config0 tiny T=256 512->512 r8 s2", 1: "config1 q_proj T=8192 4096->4096 r16 s2",
            2: "config2 gate/up_proj T=16384 4096->14336 r16 s2", 3: "config3 down_proj T=16384 14336->4096 r64 s0.5",
            4: "config4 seven Llama-3-8B projections T=32768 r16 s2",
            5: "paper setting: q/k/v/o adapters r32 alpha64 (s2), T=49152 (6 x 8k tokens per GPU)"}[idx]


# ----------------------------------------------------------------------------------------------------
# CPU oracle timing (reported baseline; also the --impl reference arm)
# ----------------------------------------------------------------------------------------------------
def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def sample_flops(proj, rows: int) -> float:
    return 4.0 * rows * proj.d_in * proj.d_out + 6.0 * rows * proj.r * (proj.d_in + proj.d_out)


def oracle_inputs(workload_idx: int, max_rows: int):
    """The first `max_rows` token rows of every projection of the workload, widened to float64 (full W, A, B)."""
    from paper_2503_22673_b200 import inputs
    protos = inputs.workload(workload_idx)
    rows = min(protos[0].T, max_rows)
    drawn = []
    for proj, t in inputs.draw_workload(workload_idx, seed=0, T=rows):
        drawn.append((proj, {k: inputs.bf16_to_f64(v) for k, v in t.items()}))
    return protos, drawn, rows


def oracle_step_time(drawn, rows: int) -> float:
    """One oracle forward + backward of every projection on its first `rows` token rows."""
    from oracle import lora_oracle as oracle
    t0 = time.perf_counter()
    for proj, f64 in drawn:
        X, dY = f64["X"][:rows], f64["dY"][:rows]
        oracle.forward(X, f64["W"], f64["A"], f64["B"], proj.scale)
        oracle.backward(dY, X, f64["W"], f64["A"], f64["B"], proj.scale)
    return time.perf_counter() - t0


def pick_rows(drawn, avail: int, budget_s: float) -> int:
    cal = min(avail, 128)
    t_cal = oracle_step_time(drawn, cal)                  # calibration (also warms the BLAS pool)
    t_cal = min(t_cal, oracle_step_time(drawn, cal))
    rows = int(budget_s / max(t_cal / cal, 1e-9))
    return min(avail, max(cal, rows - rows % 128))


def cpu_baseline(workload_idx: int, budget_s: float = 12.0):
    protos, drawn, avail = oracle_inputs(workload_idx, 2048 if len(inputs_workload(workload_idx)) > 1 else 4096)
    rows = pick_rows(drawn, avail, budget_s)
    t = oracle_step_time(drawn, rows)
    flops = sum(sample_flops(p, rows) for p in protos)
    names = "+".join(p.name for p in protos)
    return {"value": flops / t / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{names}: {rows} of {protos[0].T} token rows of every projection, full W/A/B, fp64 numpy, one fwd+bwd in {t:.2f} s",
            "tokens_per_s": rows / t}


def inputs_workload(idx):
    from paper_2503_22673_b200 import inputs
    return inputs.workload(idx)


def run_reference(args):
    rank, _, _ = dist_env()
    if rank != 0:
        return
    protos, drawn, avail = oracle_inputs(args.workload, 2048 if len(inputs_workload(args.workload)) > 1 else 4096)
    total_steps = max(args.steps + args.warmup, 1)
    rows = pick_rows(drawn, avail, min(3.0, 100.0 / total_steps))
    for _ in range(args.warmup):
        oracle_step_time(drawn, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step_time(drawn, rows)
    dt = time.perf_counter() - t0
    flops = sum(sample_flops(p, rows) for p in protos)
    value = flops * args.steps / dt / 1e12
    sample = (f"{'+'.join(p.name for p in protos)}: {rows} of {protos[0].T} token rows of every projection per step, "
              "full W/A/B, fp64 numpy")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "projections": [p.name for p in protos], "T": protos[0].T,
                   "r": protos[0].r, "scale": protos[0].scale, "sampled_rows_per_step": rows},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "tokens_per_s": rows * args.steps / dt, "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------------
# CUDA path
# ----------------------------------------------------------------------------------------------------
def to_dev(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


class Workload:
    """Device tensors, plans and the step function of one workload (n_sets independent input/output sets, rotated per step)."""

    def __init__(self, idx: int, rank: int, local_rank: int, device, n_sets: int = None, tokens: int = None):
        from paper_2503_22673_b200 import binding, inputs
        self.idx, self.device, self.binding = idx, device, binding
        self.protos = inputs.workload(idx, tokens)
        self.bytes_per_set = sum(2 * (p.T * p.d_in * 2 + p.T * p.d_out * 2) + 2 * p.d_out * p.d_in for p in self.protos)
        if n_sets is None:
            n_sets = 2 if idx >= 2 else max(2, min(6, -(-4 * L2_BYTES // self.bytes_per_set)))
        self.n_sets = n_sets
        self.sets = []
        for s_i in range(n_sets):
            cur, x_dev = [], {}
            for proj, t in inputs.draw_workload(idx, seed=1000 * rank + s_i, T=tokens):
                d = {k: to_dev(v, device) for k, v in t.items() if k != "X"}
                if proj.x_group not in x_dev:                 # projections that share X (q/k/v, gate/up) share the tensor
                    x_dev[proj.x_group] = to_dev(t["X"], device)
                d["X"] = x_dev[proj.x_group]
                d["Y"] = torch.empty((proj.T, proj.d_out), dtype=torch.bfloat16, device=device)
                d["dX"] = torch.empty((proj.T, proj.d_in), dtype=torch.bfloat16, device=device)
                d["dA"] = torch.empty((proj.r, proj.d_in), dtype=torch.float32, device=device)
                d["dB"] = torch.empty((proj.d_out, proj.r), dtype=torch.float32, device=device)
                cur.append((proj, d))
            self.sets.append(cur)
        self.plans = [binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r, device=local_rank) for p in self.protos]
        for pl in self.plans:
            pl.ensure_workspace()
        self.flops_step = float(sum(p.flops for p in self.protos))
        self.tokens_step = self.protos[0].T
        self.stage_names = [("fwd_stage",) + pl.bwd_stage_names() for pl in self.plans]

    def step(self, k, events=None, saved_p=False):
        cur = self.sets[k % self.n_sets]
        for j, (proj, d) in enumerate(cur):
            pl = self.plans[j]
            if events is None:       # the product path: lora_linear_fwd + lora_linear_bwd
                pl.fwd(d["X"], d["W"], d["A"], d["B"], proj.scale, d["Y"])
                pl.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"], saved_p=saved_p)
            else:                    # the same launches through the stage calls, with an event before and after each stage
                ev = events[j]
                ev[0].record()
                pl.fwd(d["X"], d["W"], d["A"], d["B"], proj.scale, d["Y"])
                pl.bwd_stages(d["dY"], d["X"], d["W"], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"], events=ev[1:])

    def check_status(self, where):
        for pl in self.plans:
            code, msg = pl.device_status()
            if code != 0:
                raise SystemExit(f"bench.py: device status {where}: {msg}")

    def close(self):
        for pl in self.plans:
            pl.close()
        self.sets = []
        import gc
        gc.collect()
        torch.cuda.empty_cache()


def stage_bytes(p, stage: str) -> float:
    """Algorithmic bytes of one launch (group) of the skinny stages: the streamed matrices once, the small factors, the result."""
    x, dy = 2.0 * p.T * p.d_in, 2.0 * p.T * p.d_out
    small_t = 2.0 * p.T * p.r                      # one [r, T] bf16 factor
    return {"sides": x + dy + 2 * small_t + 2.0 * p.r * (p.d_in + p.d_out),
            "grads": x + dy + 2 * small_t + 4.0 * p.r * (p.d_in + p.d_out),
            "q_prepass": dy + small_t + 2.0 * p.r * p.d_out,
            "dA": x + 2 * small_t + 4.0 * p.r * p.d_in,
            "dB": dy + small_t + 4.0 * p.r * p.d_out}[stage]


def measure(wl: Workload, steps: int, warmup: int, pk, world: int, device, barrier, sampler=None):
    """Timed region (K steps back to back between two events) and the instrumented pass (events between the stages)."""
    binding = wl.binding
    n_warm = max(warmup, 3)
    for k in range(n_warm):
        wl.step(k)
    torch.cuda.synchronize()
    wl.check_status("after warm-up")
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the same steps timed straight after the W warm-up steps, before the part has settled: reported beside the headline as
    # `ms_per_step_cold_start`, never as the value
    c_a, c_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_cold = min(steps, 20)
    c_a.record()
    for k in range(n_cold):
        wl.step(n_warm + k)
    c_b.record()
    torch.cuda.synchronize()
    ms_cold = c_a.elapsed_time(c_b) / max(n_cold, 1)
    # once more, and on until the part has been under load for SETTLE_S seconds: after a cold start the power controller
    # first lets the clock overshoot and then clamps it for about a second; the timed region should see neither
    t_settle, n_settle = time.time(), 0
    while n_settle < n_warm or (time.time() - t_settle < SETTLE_S and n_settle < 400):
        wl.step(n_settle)
        n_settle += 1
        if n_settle % 4 == 0:
            torch.cuda.synchronize()     # keeps the host clock in step with the device
    n_warm_total = n_warm + n_settle
    launches0 = binding.launch_count()
    barrier()
    torch.cuda.synchronize()
    t_host0 = time.time()
    ev_a.record()
    for k in range(steps):
        wl.step(n_warm + k)
    ev_b.record()
    torch.cuda.synchronize()
    t_host1 = time.time()
    barrier()
    launches = binding.launch_count() - launches0
    ms_step = max_over_ranks(ev_a.elapsed_time(ev_b), device, world) / steps
    # SM clock of the last GEMM launch of every projection, measured inside the kernel
    gemm_clock = {p.name: round(pl.last_gemm_clock()[0], 1) for p, pl in zip(wl.protos, wl.plans)}

    # ---- the same steps once more with events between the stages: per-stage durations.  An event record between two
    #      launches suppresses their programmatic overlap, so this pass is a little slower than the timed region ----
    n_instr = min(steps, 20)
    events = [[[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for names in wl.stage_names]
              for _ in range(n_instr)]
    i_a, i_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    i_a.record()
    for k in range(n_instr):
        wl.step(n_warm + k, events[k])
    i_b.record()
    torch.cuda.synchronize()
    t_host2 = time.time()
    ms_step_instr = i_a.elapsed_time(i_b) / n_instr
    wl.check_status("after the timed region")

    kern = {}
    for j, p in enumerate(wl.protos):
        names = wl.stage_names[j]
        dur = [statistics.mean(events[k][j][i].elapsed_time(events[k][j][i + 1]) for k in range(n_instr)) for i in range(len(names))]
        cfg = wl.plans[j].config()
        entry = {}
        for name, ms in zip(names, dur):
            if name == "fwd_stage":
                fl = 2.0 * p.T * p.d_in * p.d_out + 2.0 * p.T * p.r * (p.d_in + p.d_out)
                entry[name] = {"ms": ms, "tflops": fl / ms / 1e9, "frac_of_bf16_peak": fl / ms / 1e9 / pk["bf16_tflops"],
                               "launches": "X A^T pass + K-extended GEMM" if cfg["fwd_ext"] and cfg["cta_group"] == 2 else "fused GEMM"}
            elif name == "dx_gemm":
                fl = 2.0 * p.T * p.d_in * p.d_out + 2.0 * p.T * p.r * p.d_in          # dense + the rank-r k-block (Q A)
                entry[name] = {"ms": ms, "tflops": fl / ms / 1e9, "frac_of_bf16_peak": fl / ms / 1e9 / pk["bf16_tflops"],
                               "frac_of_bf16_sustained": fl / ms / 1e9 / pk["bf16_tflops_sustained"]}
            else:
                by = stage_bytes(p, name)
                entry[name] = {"ms": ms, "gbs": by / ms / 1e6, "frac_of_hbm_peak": by / ms / 1e6 / pk["hbm_gbs"],
                               "bytes": by}
        kern[p.name] = entry
    return {"ms_per_step": ms_step, "ms_per_step_instrumented": ms_step_instr, "launches": launches, "kernels": kern,
            "gemm_sm_mhz_in_kernel": gemm_clock, "t_host": (t_host0, t_host1, t_host2), "n_warm": n_warm_total + n_cold, "ms_per_step_cold_start": ms_cold}


def copy_behind_gemms(wl: Workload, nbytes: float, device, n: int = 6) -> float:
    """GB/s of a plain device-to-device copy that moves `nbytes` (half read, half written), timed between two events right
    after a whole step of the workload, n times.  Context for the HBM fractions only: the copy is torch's own kernel, and it
    shows what a streaming launch can reach at the clocks the power-capped GEMMs leave behind (the measured copy peak in
    MEASURED_PEAKS.json was taken on an otherwise idle part)."""
    elems = int(nbytes // 4)                           # bf16: nbytes / 2 bytes each way
    src = [torch.empty(elems, dtype=torch.bfloat16, device=device).normal_() for _ in range(2)]
    dst = torch.empty(elems, dtype=torch.bfloat16, device=device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for k in range(n):
        wl.step(k)
        ev[k][0].record()
        dst.copy_(src[k % 2])
        ev[k][1].record()
    torch.cuda.synchronize()
    ms = statistics.mean(a.elapsed_time(b) for a, b in ev)
    del src, dst
    return 4.0 * elems / ms / 1e6


def kernel_b2b(wl: Workload, pk, n: int = 16):
    """Every skinny stage of every projection launched n times back to back (inputs rotate between the sets, so the
    stream never sits in L2): the launch's own steady-state duration, with the programmatic overlap of consecutive
    launches that the step itself enjoys and the instrumented pass suppresses."""
    out = {}
    for j, p in enumerate(wl.protos):
        pl = wl.plans[j]
        lib, h = pl._lib, pl._h
        from paper_2503_22673_b200.binding import _ptr, _stream_ptr
        sp = _stream_ptr(None)
        res = {}
        for name in pl.bwd_stage_names():
            if name == "dx_gemm":
                continue

            def call(k, name=name):
                d = wl.sets[k % wl.n_sets][j][1]
                s = float(p.scale)
                if name == "sides":
                    return lib.lora_linear_bwd_sides(h, _ptr(d["dY"]), _ptr(d["X"]), _ptr(d["A"]), _ptr(d["B"]), s, sp)
                if name == "grads":
                    return lib.lora_linear_bwd_grads(h, _ptr(d["dY"]), _ptr(d["X"]), _ptr(d["A"]), s, _ptr(d["dA"]), _ptr(d["dB"]), sp)
                if name == "q_prepass":
                    return lib.lora_linear_bwd_q(h, _ptr(d["dY"]), _ptr(d["B"]), s, sp)
                if name == "dA":
                    return lib.lora_linear_bwd_da(h, _ptr(d["X"]), _ptr(d["A"]), s, _ptr(d["dA"]), sp)
                return lib.lora_linear_bwd_db(h, _ptr(d["dY"]), s, _ptr(d["dB"]), sp)

            for k in range(3):
                call(k)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for k in range(n):
                call(3 + k)
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b) / n
            by = stage_bytes(p, name)
            res[name] = {"ms": ms, "gbs": by / ms / 1e6, "frac_of_hbm_peak": by / ms / 1e6 / pk["hbm_gbs"]}
        out[p.name] = res
    return out


def graph_replay_ms(wl: Workload, steps: int) -> float:
    """ms per step when every input set's step is captured into a CUDA graph once and the graphs are replayed in rotation."""
    graphs = []
    for k in range(wl.n_sets):
        wl.step(k)                                   # eager once: nothing is left to initialise inside the capture
    torch.cuda.synchronize()
    for k in range(wl.n_sets):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            wl.step(k)
        graphs.append(g)
    for k in range(2 * wl.n_sets):
        graphs[k % wl.n_sets].replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for k in range(steps):
        graphs[k % wl.n_sets].replay()
    b.record()
    torch.cuda.synchronize()
    wl.check_status("after the graph replays")
    del graphs
    return a.elapsed_time(b) / steps


def timed_loop(fn, n, barrier, device, world):
    for k in range(3):
        fn(k)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    a.record()
    for k in range(n):
        fn(3 + k)
    b.record()
    torch.cuda.synchronize()
    barrier()
    return max_over_ranks(a.elapsed_time(b) / n, device, world)


def run_ours(args):
    from paper_2503_22673_b200 import binding
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device - the layer has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    pk = peaks()
    # nvidia-smi takes a while to start: launch it now, keep the samples whose timestamps fall into the timed regions
    sampler = ClockSampler(local_rank) if rank == 0 else None

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    wl = Workload(args.workload, rank, local_rank, device, tokens=args.tokens)
    protos, plans = wl.protos, wl.plans
    m = measure(wl, args.steps, args.warmup, pk, world, device, barrier)
    ms_step, kern = m["ms_per_step"], m["kernels"]
    flops_step, tokens_step = wl.flops_step, wl.tokens_step

    # ---- sustained leg: the same step looped back to back for at least two seconds (clock samples inside it) ----
    n_sus = max(args.steps, int(2200.0 / ms_step) + 1) if not args.quick else args.steps
    s_a, s_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    t_sus0 = time.time()
    s_a.record()
    for k in range(n_sus):
        wl.step(k)
    s_b.record()
    torch.cuda.synchronize()
    t_sus1 = time.time()
    barrier()
    ms_sus = max_over_ranks(s_a.elapsed_time(s_b), device, world) / n_sus
    sus_clock = {p.name: round(pl.last_gemm_clock()[0], 1) for p, pl in zip(protos, plans)}
    b2b = kernel_b2b(wl, pk)
    clocks_raw = sampler.stop(*m["t_host"][:2]) if sampler is not None else None
    clocks = clocks_raw
    sus_clocks = sampler.window(t_sus0, t_sus1, "sustained leg") if sampler is not None else None

    # dominant kernel for the roofline: the dX GEMM launch of the projection with the longest GEMMs (its event pair
    # brackets exactly ONE kernel: the K-extended CTA-pair GEMM; the skinny launch that feeds it sits before the first event)
    dom_p = max(protos, key=lambda p: kern[p.name]["fwd_stage"]["ms"] + kern[p.name]["dx_gemm"]["ms"])
    dom_plan = plans[protos.index(dom_p)].config()
    dom = kern[dom_p.name]["dx_gemm"]
    dx_launches = 1 + (1 if dom_plan["dx_split_k"] > 1 and dom_plan["cta_group"] == 2 else 0)
    gemm_key = f"{dom_p.T}x{dom_p.d_in}x{dom_p.d_out}"
    roofline = {"bound": "tensor",
                "kernel": f"lora_gemm_pair_kernel<1,1>: dX = dY W + (s dY B) A as one K-extended GEMM ({dom_p.name}, {gemm_key})"
                          if dom_plan["cta_group"] == 2 else f"lora_gemm_kernel<1> (single-CTA dX GEMM, {dom_p.name})",
                "launches_in_bracket": dx_launches,
                "achieved": dom["tflops"], "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": dom["tflops"] / pk["bf16_tflops_sustained"],
                "peak_kind": f"bf16 sustained (the kernel is timed inside a long step), of {pk['source']}",
                "frac_of_burst": dom["tflops"] / pk["bf16_tflops"], "burst_peak": pk["bf16_tflops"],
                "sm_mhz_in_kernel": m["gemm_sm_mhz_in_kernel"].get(dom_p.name),
                "ms_per_launch": dom["ms"],
                "flops_per_launch": 2.0 * dom_p.T * dom_p.d_in * dom_p.d_out + 2.0 * dom_p.T * dom_p.r * dom_p.d_in,
                "traffic": (NCU_TRAFFIC["gemm_bytes_per_launch"].get(gemm_key)
                            if NCU_TRAFFIC["gemm_sha"] == source_sha("gemm") else None)}
    # the skinny stage furthest below the HBM roofline (stage = one launch; duration between the events around it)
    worst = None
    for p in protos:
        for name, e in kern[p.name].items():
            if "frac_of_hbm_peak" in e and (worst is None or e["frac_of_hbm_peak"] < worst[2]["frac_of_hbm_peak"]):
                worst = (p, name, e)
    roofline_hbm = None
    if worst is not None:
        wp, wname, we = worst
        skey = f"{wname}:{wp.T}x{wp.d_in}x{wp.d_out}"
        roofline_hbm = {"bound": "hbm", "kernel": f"lora_grad_kernel, stage '{wname}' of {wp.name} ({wp.T} x {wp.d_in} -> {wp.d_out})",
                        "achieved": we["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": we["frac_of_hbm_peak"],
                        "peak_kind": f"STREAM-style copy, of {pk['source']}", "ms_per_launch": we["ms"], "bytes_per_launch": we["bytes"],
                        "back_to_back": b2b.get(wp.name, {}).get(wname),
                        "traffic": (NCU_TRAFFIC["stream_bytes_per_launch"].get(skey)
                                    if NCU_TRAFFIC["stream_sha"] == source_sha("adapter_grad") else None)}
        if not args.quick:
            cg = copy_behind_gemms(wl, we["bytes"], device)
            roofline_hbm["plain_copy_same_bytes_behind_gemms"] = {
                "gbs": cg, "frac_of_hbm_peak": cg / pk["hbm_gbs"],
                "note": "a device-to-device copy (torch's kernel, measurement only) moving the stage's byte count, between two "
                        "events right after a whole step: the copy rate at the clocks the power-capped GEMMs leave behind"}

    variants = {}
    n_var = max(3, min(args.steps, 20))
    if not args.quick:
        # ---- variant: backward that reuses the forward's X A^T (lora_linear_bwd_saved_p), same inputs and rotation ----
        ms_var = timed_loop(lambda k: wl.step(k, saved_p=True), n_var, barrier, device, world)
        variants["bwd_saved_p"] = {"ms_per_step": ms_var, "value": job_value(world, flops_step, ms_var), "unit": UNIT,
                                   "steps": n_var, "note": "forward + lora_linear_bwd_saved_p (X A^T kept from the forward)"}
        # ---- variant: quantised LoRA (NF4 frozen weight): lora_linear_fwd_nf4 + lora_linear_bwd_nf4, same inputs.  Two forms:
        #      weight expanded once per call into a scratch buffer (fast), or expanded inside the GEMM kernels (no extra memory)
        if all(p.d_in % 64 == 0 for p in protos):
            q_sets = [[binding.nf4_quantize(d["W"]) for _, d in cur] for cur in wl.sets]
            w_scratch = {}
            for p in protos:
                if (p.d_out, p.d_in) not in w_scratch:
                    w_scratch[(p.d_out, p.d_in)] = torch.empty((p.d_out, p.d_in), dtype=torch.bfloat16, device=device)

            band = None
            if all(p.T > 128 for p in protos):
                band_bytes = max(NF4_BAND_BYTES, max(pl.nf4_scratch_bytes()[0] for pl in plans))
                band = torch.empty((band_bytes // 2,), dtype=torch.bfloat16, device=device)   # ONE buffer for every projection

            def step_nf4(k, scratch):
                cur, qs = wl.sets[k % wl.n_sets], q_sets[k % wl.n_sets]
                for j, (proj, d) in enumerate(cur):
                    ws = band if scratch == "band" else w_scratch[(proj.d_out, proj.d_in)] if scratch else None
                    plans[j].fwd_nf4(d["X"], qs[j][0], qs[j][1], d["A"], d["B"], proj.scale, d["Y"], w_scratch=ws)
                    plans[j].bwd_nf4(d["dY"], d["X"], qs[j][0], qs[j][1], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"],
                                     w_scratch=ws)

            forms = [("q_lora_nf4", True, "weight expanded once per call into a bf16 scratch buffer, then the bf16 kernels")]
            if band is not None:
                forms.append(("q_lora_nf4_banded", "band", f"one {band.numel() * 2 >> 20} MiB scratch buffer for all projections: the "
                              "weight is expanded and multiplied band by band (bands of output features forward, of input features backward)"))
                forms.append(("q_lora_nf4_in_kernel", False, "no scratch: weight expanded inside the GEMM kernels, per 256-token tile"))
            for key, scratch, how in forms:
                ms_q = timed_loop(lambda k: step_nf4(k, scratch), n_var, barrier, device, world)
                variants[key] = {"ms_per_step": ms_q, "value": job_value(world, flops_step, ms_q), "unit": UNIT, "steps": n_var,
                                 "tokens_per_s": world * tokens_step / ms_q * 1e3,
                                 "note": "forward + backward with the frozen W in NF4 (4.5 bits per weight); " + how +
                                         "; same algorithmic FLOPs as the bf16 step"}
            del q_sets, w_scratch, band
        # ---- variant: projections that share X (q/k/v, gate/up) through the grouped calls, the others through their own plans ----
        group_ids = {4: [[0, 1, 2], [4, 5]], 5: [[0, 1, 2]]}.get(args.workload, [])
        if group_ids and all(p.r % 16 == 0 for p in protos):
            from paper_2503_22673_b200.grouped import GroupedLoraPlan
            grouped, in_group = [], set()
            for ids in group_ids:
                in_group.update(ids)
                p0 = protos[ids[0]]
                gp = GroupedLoraPlan(p0.T, p0.d_in, [protos[i].d_out for i in ids], p0.r, device=local_rank)
                per_set = []
                for cur in wl.sets:
                    W, A, B = gp.pack([cur[i][1]["W"] for i in ids], [cur[i][1]["A"] for i in ids], [cur[i][1]["B"] for i in ids])
                    dYc = torch.cat([cur[i][1]["dY"] for i in ids], dim=1).contiguous()
                    per_set.append({"X": cur[ids[0]][1]["X"], "W": W, "A": A, "B": B, "dY": dYc,
                                    "Y": torch.empty_like(dYc), "dX": torch.empty_like(cur[ids[0]][1]["X"]),
                                    "dA": torch.empty((gp.G * gp.r, gp.d_in), dtype=torch.float32, device=device),
                                    "dB": torch.empty((gp.D, gp.r), dtype=torch.float32, device=device)})
                grouped.append((gp, p0.scale, per_set))
            singles = [j for j in range(len(protos)) if j not in in_group]

            def step_grouped(k):
                for gp, sc, per_set in grouped:
                    d = per_set[k % wl.n_sets]
                    gp.fwd(d["X"], d["W"], d["A"], d["B"], sc, d["Y"])
                    gp.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], sc, d["dX"], d["dA"], d["dB"])
                cur = wl.sets[k % wl.n_sets]
                for j in singles:
                    proj, d = cur[j]
                    plans[j].fwd(d["X"], d["W"], d["A"], d["B"], proj.scale, d["Y"])
                    plans[j].bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"])

            ms_g = timed_loop(step_grouped, n_var, barrier, device, world)
            for gp, _, _ in grouped:
                code, msg = gp.device_status()
                if code != 0:
                    raise SystemExit(f"bench.py: device status after the grouped variant: {msg}")
            variants["grouped_shared_x"] = {
                "ms_per_step": ms_g, "value": job_value(world, flops_step, ms_g), "unit": UNIT, "steps": n_var,
                "tokens_per_s": world * tokens_step / ms_g * 1e3,
                "note": "projections sharing X through lora_linear_fwd_grouped / lora_linear_bwd_grouped ("
                        + ", ".join("+".join(protos[i].name for i in ids) for ids in group_ids)
                        + "), the others through their own plans; same algorithmic FLOPs (dX of a group is one sum)"}
            for gp, _, _ in grouped:
                gp.close()
            del grouped
        # ---- extra kernel: the dense weight gradient of full fine-tuning, dW = dY^T X (lora_dense_dw), per projection ----
        dw_out = [torch.empty((p.d_out, p.d_in), dtype=torch.bfloat16, device=device) for p in protos]

        def step_dw(k):
            for j, (proj, d) in enumerate(wl.sets[k % wl.n_sets]):
                plans[j].dense_dw(d["dY"], d["X"], dw_out[j])

        ms_dw = timed_loop(step_dw, n_var, barrier, device, world)
        dw_flops = float(sum(2.0 * p.T * p.d_in * p.d_out for p in protos))
        variants["full_ft_dense_dw"] = {"ms_per_step": ms_dw, "value": job_value(world, dw_flops, ms_dw), "unit": UNIT,
                                        "frac_of_bf16_peak": dw_flops / ms_dw / 1e9 / pk["bf16_tflops"], "steps": n_var,
                                        "note": "lora_dense_dw alone (dW = dY^T X, 2 T d_in d_out FLOPs per projection); not part "
                                                "of the LoRA step"}
        del dw_out

    # ---- end to end: host buffers through the C ABI (lora_linear_step_host), copies inside the timed region.  Every step
    #      copies its inputs from pinned host memory, runs forward + backward and copies Y, dX, dA, dB back.  Two lanes
    #      (plan + staging + host output buffers + stream each) alternate, so that the copy-in of one step overlaps the
    #      copy-out of the previous one on the two DMA directions; each step's own chain stays in order on its stream ----
    e2e = None
    if not args.quick:
        n_lanes = 1 if args.workload >= 4 else 2
        sets0 = wl.sets[0]
        h_in = [{k: d0[k].cpu().pin_memory() for k in ("X", "A", "B", "dY")} for _, d0 in sets0]
        lanes = []
        for ln in range(n_lanes):
            lp = plans if ln == 0 else [binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r, device=local_rank) for p in protos]
            for pl in lp:
                pl.ensure_workspace()
            outs = [{k: torch.empty_like(d0[k], device="cpu").pin_memory() for k in ("Y", "dX", "dA", "dB")} for _, d0 in sets0]
            stg = [torch.empty(lp[j].step_host_staging_bytes(), dtype=torch.uint8, device=device) for j in range(len(protos))]
            # a lane with several projections (each with its own plan, staging and host buffers) runs them on E2E_STREAMS
            # streams in turn, so that one projection's copy-out overlaps the next ones' copy-in within the step as well
            n_streams = min(E2E_STREAMS, len(protos))
            lanes.append({"plans": lp, "out": outs, "staging": stg,
                          "streams": [torch.cuda.Stream(device=device) for _ in range(n_streams)]})

        def step_host(k):
            ln = lanes[k % n_lanes]
            for j, (p, d0) in enumerate(sets0):
                h, ho = h_in[j], ln["out"][j]
                ln["plans"][j].step_host(h["X"], d0["W"], h["A"], h["B"], h["dY"], p.scale, ho["Y"], ho["dX"], ho["dA"], ho["dB"],
                                         ln["staging"][j], stream=ln["streams"][j % len(ln["streams"])])

        def run_host(n):
            cur = torch.cuda.current_stream()
            start, done = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record(cur)
            for ln in lanes:
                for st in ln["streams"]:
                    st.wait_event(start)
            for k in range(n):
                step_host(k)
            for ln in lanes:
                for st in ln["streams"]:
                    ev = torch.cuda.Event()
                    ev.record(st)
                    cur.wait_event(ev)
            done.record(cur)
            torch.cuda.synchronize()
            return start.elapsed_time(done)

        n_e2e = max(3, min(args.steps, 20 if args.workload < 4 else 3))
        run_host(2 * n_lanes if args.workload < 4 else 1)
        barrier()
        ms_e2e = max_over_ranks(run_host(n_e2e) / n_e2e, device, world)
        barrier()
        h2d = sum(t.numel() * t.element_size() for h in h_in for t in h.values())
        d2h = sum(t.numel() * t.element_size() for ho in lanes[0]["out"] for t in ho.values())
        e2e = {"value": job_value(world, flops_step, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": ms_e2e, "steps": n_e2e, "lanes": n_lanes,
               "pcie_gbs": {"h2d": h2d / ms_e2e / 1e6, "d2h": d2h / ms_e2e / 1e6},
               "note": "host X, A, B, dY in; Y, dX, dA, dB out (pinned); frozen W resident on the device; "
                       f"{n_lanes} lane(s) of lora_linear_step_host alternate so that copies of neighbouring steps overlap"
                       + (f"; the projections of a step rotate over {min(E2E_STREAMS, len(protos))} streams" if len(protos) > 1 else "")}
    plan_desc = plans[0].describe()
    wl.close()

    # ---- the other workloads, from short runs in the same process (rank 0's figures; every rank runs them) ----
    per_config = {}
    if not args.quick and world == 1:
        for idx in [i for i in (0, 1, 2, 3, 4, 5) if i != args.workload]:
            w2 = Workload(idx, rank, local_rank, device)
            k2 = {0: 200, 1: 100, 2: 20, 3: 20, 4: 5, 5: 10}[idx]
            m2 = measure(w2, k2, 3, pk, world, device, barrier)
            v2 = job_value(1, w2.flops_step, m2["ms_per_step"])
            stages = {}
            for pn, e in m2["kernels"].items():
                stages[pn] = {sn: ({"us": round(se["ms"] * 1e3, 1), "frac_of_hbm_peak": round(se["frac_of_hbm_peak"], 3)}
                                   if "frac_of_hbm_peak" in se else
                                   {"us": round(se["ms"] * 1e3, 1), "tflops": round(se["tflops"], 1)}) for sn, se in e.items()}
            b2 = kernel_b2b(w2, pk)
            graph_ms = graph_replay_ms(w2, k2) if m2["ms_per_step"] < 0.1 else None      # launch-bound steps only
            cp_bytes = stage_bytes(w2.protos[0], "sides")
            cp_gbs = copy_behind_gemms(w2, cp_bytes, device) if idx != 0 else None
            per_config[f"workload{idx}"] = {
                "workload": workload_name(idx), "steps": k2, "ms_per_step": m2["ms_per_step"], "tflops": v2,
                "ms_per_step_cold_start": m2["ms_per_step_cold_start"],
                "tflops_cold_start": job_value(1, w2.flops_step, m2["ms_per_step_cold_start"]),
                "tokens_per_s": w2.tokens_step / m2["ms_per_step"] * 1e3,
                "frac_of_bf16_burst": v2 / pk["bf16_tflops"], "frac_of_bf16_sustained": v2 / pk["bf16_tflops_sustained"],
                "gemm_sm_mhz_in_kernel": m2["gemm_sm_mhz_in_kernel"], "stages": stages,
                "skinny_back_to_back": {pn: {sn: {"us": round(se["ms"] * 1e3, 1), "frac_of_hbm_peak": round(se["frac_of_hbm_peak"], 3)}
                                             for sn, se in e.items()} for pn, e in b2.items()},
                "input_sets_rotated": w2.n_sets}
            if cp_gbs is not None:
                per_config[f"workload{idx}"]["plain_copy_sides_bytes_behind_gemms"] = {
                    "bytes": cp_bytes, "gbs": round(cp_gbs, 1), "frac_of_hbm_peak": round(cp_gbs / pk["hbm_gbs"], 3),
                    "note": "torch copy kernel moving the sides stage's byte count, between two events after a step (context only)"}
            if graph_ms is not None:
                per_config[f"workload{idx}"]["cuda_graph_replay"] = {
                    "ms_per_step": graph_ms, "tflops": job_value(1, w2.flops_step, graph_ms),
                    "note": "the same step (lora_linear_fwd + lora_linear_bwd) captured once per input set into a CUDA graph and "
                            "replayed: the calls only enqueue work, so the host's launch cost drops out"}
            w2.close()

    if rank != 0:
        return
    cpu = cpu_baseline(args.workload) if world == 1 and not args.no_cpu_baseline else None
    value = job_value(world, flops_step, ms_step)
    v_sus = job_value(world, flops_step, ms_sus)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": m["n_warm"],
        "ms_per_step": ms_step, "ms_per_step_instrumented": m["ms_per_step_instrumented"],
        "ms_per_step_cold_start": m["ms_per_step_cold_start"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "projections": [p.name for p in protos], "T": protos[0].T,
                   "r": protos[0].r, "scale": protos[0].scale, "input_sets_rotated": wl.n_sets,
                   "l2": f"{wl.n_sets} independent input/output sets ({wl.bytes_per_set * wl.n_sets / 2**20:.0f} MiB) rotated per step; "
                         "each step's operands exceed the 126 MB L2",
                   "replicas": "independent replica per GPU, no collective"},
        "tokens_per_s": world * tokens_step / ms_step * 1e3,
        "frac_of_bf16_peak": value / world / pk["bf16_tflops"], "frac_of_bf16_sustained_peak": value / world / pk["bf16_tflops_sustained"],
        "peak_source": pk["source"], "peaks": {k: pk[k] for k in ("bf16_tflops", "bf16_tflops_sustained", "hbm_gbs")},
        "sustained": {"value": v_sus, "unit": UNIT, "ms_per_step": ms_sus, "steps": n_sus, "seconds": ms_sus * n_sus / 1e3,
                      "tokens_per_s": world * tokens_step / ms_sus * 1e3,
                      "frac_of_bf16_burst": v_sus / world / pk["bf16_tflops"], "frac_of_bf16_sustained": v_sus / world / pk["bf16_tflops_sustained"],
                      "gemm_sm_mhz_in_kernel": sus_clock, "clocks": sus_clocks},
        "gemm_sm_mhz_in_kernel": m["gemm_sm_mhz_in_kernel"],
        "kernels": kern, "skinny_back_to_back": b2b, "variants": variants, "roofline": roofline, "roofline_hbm": roofline_hbm,
        "per_config": per_config, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": m["launches"], "clocks": clocks,
        "plan": plan_desc,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tokens", type=int, default=None,
                    help="override the workload's token count (profiler captures of a kernel at a size small enough to capture; "
                         "the line's config then names the reduced T)")
    ap.add_argument("--quick", action="store_true",
                    help="only the timed region and the instrumented pass of the chosen workload (no sustained leg, variants, "
                         "end-to-end leg or other workloads); for profiler captures")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

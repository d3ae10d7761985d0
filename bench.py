#!/usr/bin/env python
"""Throughput of the LoRA projection layer (forward + backward) on B200.

A step is one pass of the whole hot path - forward GEMM with the fused adapter, dX GEMM with the fused
adapter, dA kernel, dB kernel - over one batch of seeded synthetic input.  The default workload is the
Llama-3-8B q_proj shape (T = 8192 packed tokens, 4096 -> 4096, r = 16, s = 2).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload {0..4}] [--impl reference]

Prints ONE JSON line.  With N > 1 (torchrun, one rank per GPU) every rank runs an independent replica
on its own batch: the layer has no collective, so the job's value is the sum over ranks divided by the
slowest rank's time.
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
METRIC = "lora_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel from an
# ncu capture summarised under profiles/; only valid for the kernel source it was taken on.
NCU_TRAFFIC = {"gemm_sha": "7c3994e03b7d900f", "bytes_per_launch": {"fwd_gemm": 221.3e6, "dx_gemm": 219.7e6}}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def gemm_source_sha() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2503_22673_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.startswith("gemm") or name in ("sm100_ptx.cuh", "kernels.h"):
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
        inside = [r for r in rows if t0 is not None and r[0] is not None and t0 <= r[0] <= t1]
        window = "timed region" if inside else "whole run (no sample fell inside the timed region)"
        use = inside if inside else rows
        sm = [r[1] for r in use]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(r[2] for r in use) if use else None,
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


def oracle_step_time(proj, f64, rows: int) -> float:
    """One oracle forward + backward on the first `rows` token rows (all of W, A, B)."""
    from oracle import lora_oracle as oracle
    X, dY = f64["X"][:rows], f64["dY"][:rows]
    t0 = time.perf_counter()
    oracle.forward(X, f64["W"], f64["A"], f64["B"], proj.scale)
    oracle.backward(dY, X, f64["W"], f64["A"], f64["B"], proj.scale)
    return time.perf_counter() - t0


def sample_flops(proj, rows: int) -> float:
    return 4.0 * rows * proj.d_in * proj.d_out + 6.0 * rows * proj.r * (proj.d_in + proj.d_out)


def oracle_inputs(workload_idx: int, max_rows: int):
    from paper_2503_22673_b200 import inputs
    proto = inputs.workload(workload_idx)[0]
    rows = min(proto.T, max_rows)
    proj, t = next(iter(inputs.draw_workload(workload_idx, seed=0, T=rows)))
    f64 = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    return proto, proj, f64, rows


def pick_rows(proj, f64, avail: int, budget_s: float) -> int:
    cal = min(avail, 128)
    t_cal = oracle_step_time(proj, f64, cal)              # calibration (also warms the BLAS pool)
    t_cal = min(t_cal, oracle_step_time(proj, f64, cal))
    rows = int(budget_s / max(t_cal / cal, 1e-9))
    rows = min(avail, max(cal, rows - rows % 128))
    return rows


def cpu_baseline(workload_idx: int, budget_s: float = 12.0):
    proto, proj, f64, avail = oracle_inputs(workload_idx, 4096)
    rows = pick_rows(proj, f64, avail, budget_s)
    t = oracle_step_time(proj, f64, rows)
    return {"value": sample_flops(proto, rows) / t / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{proto.name}: {rows} of {proto.T} token rows, full W/A/B, fp64 numpy, one fwd+bwd in {t:.2f} s",
            "tokens_per_s": rows / t}


def run_reference(args):
    rank, _, _ = dist_env()
    if rank != 0:
        return
    proto, proj, f64, avail = oracle_inputs(args.workload, 4096)
    total_steps = max(args.steps + args.warmup, 1)
    rows = pick_rows(proj, f64, avail, min(3.0, 100.0 / total_steps))
    for _ in range(args.warmup):
        oracle_step_time(proj, f64, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step_time(proj, f64, rows)
    dt = time.perf_counter() - t0
    value = sample_flops(proto, rows) * args.steps / dt / 1e12
    sample = f"{proto.name}: {rows} of {proto.T} token rows per step, full W/A/B, fp64 numpy"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "T": proto.T, "d_in": proto.d_in, "d_out": proto.d_out,
                   "r": proto.r, "scale": proto.scale, "sampled_rows_per_step": rows},
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


def run_ours(args):
    from paper_2503_22673_b200 import binding, inputs
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device - the layer has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    pk = peaks()
    # nvidia-smi takes a while to start: launch it now, keep the samples whose timestamps fall into the timed region
    sampler = ClockSampler(local_rank) if rank == 0 else None

    # ---- inputs: n_sets independent seeded batches, rotated so that no step finds its operands in L2 ----
    protos = inputs.workload(args.workload)
    bytes_per_set = sum(2 * (p.T * p.d_in * 2 + p.T * p.d_out * 2) + 2 * p.d_out * p.d_in for p in protos)
    n_sets = max(2, min(6, -(-4 * L2_BYTES // bytes_per_set)))
    if args.workload >= 4:
        n_sets = 2
    sets = []
    for s_i in range(n_sets):
        cur = []
        for proj, t in inputs.draw_workload(args.workload, seed=1000 * rank + s_i):
            d = {k: to_dev(v, device) for k, v in t.items()}
            d["Y"] = torch.empty((proj.T, proj.d_out), dtype=torch.bfloat16, device=device)
            d["dX"] = torch.empty((proj.T, proj.d_in), dtype=torch.bfloat16, device=device)
            d["dA"] = torch.empty((proj.r, proj.d_in), dtype=torch.float32, device=device)
            d["dB"] = torch.empty((proj.d_out, proj.r), dtype=torch.float32, device=device)
            cur.append((proj, d))
        sets.append(cur)
    if args.grouped and args.workload == 4:
        # q/k/v and gate/up consume the same X: each group becomes ONE projection (stacked A, block-diagonal B)
        from paper_2503_22673_b200.grouped import GroupedLoraPlan
        groups = [[0, 1, 2], [3], [4, 5], [6]]
        new_protos, new_sets = [], [[] for _ in sets]
        for idxs in groups:
            p0 = protos[idxs[0]]
            if len(idxs) == 1:
                new_protos.append(p0)
                for si, cur in enumerate(sets):
                    new_sets[si].append(cur[idxs[0]])
                continue
            d_outs = [protos[i].d_out for i in idxs]
            gp = inputs.Projection("+".join(protos[i].name for i in idxs), p0.T, p0.d_in, sum(d_outs), p0.r * len(idxs),
                                   p0.scale)
            new_protos.append(gp)
            helper = GroupedLoraPlan(p0.T, p0.d_in, d_outs, p0.r, device=local_rank)
            for si, cur in enumerate(sets):
                W, A, B = helper.pack([cur[i][1]["W"] for i in idxs], [cur[i][1]["A"] for i in idxs],
                                      [cur[i][1]["B"] for i in idxs])
                d = {"X": cur[idxs[0]][1]["X"], "W": W, "A": A, "B": B,
                     "dY": torch.cat([cur[i][1]["dY"] for i in idxs], dim=1).contiguous()}
                d["Y"] = torch.empty((gp.T, gp.d_out), dtype=torch.bfloat16, device=device)
                d["dX"] = torch.empty((gp.T, gp.d_in), dtype=torch.bfloat16, device=device)
                d["dA"] = torch.empty((gp.r, gp.d_in), dtype=torch.float32, device=device)
                d["dB"] = torch.empty((gp.d_out, gp.r), dtype=torch.float32, device=device)
                new_sets[si].append((gp, d))
            helper.close()
        flops_algorithmic = float(sum(p.flops for p in protos))      # the seven projections' own FLOPs
        protos, sets = new_protos, new_sets
        del new_sets
        import gc
        gc.collect()
        torch.cuda.empty_cache()
    else:
        flops_algorithmic = float(sum(p.flops for p in protos))
    plans = [binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r, device=local_rank) for p in protos]
    for pl in plans:
        pl.ensure_workspace()
    flops_step = flops_algorithmic
    tokens_step = protos[0].T

    def step(k, events=None):
        cur = sets[k % n_sets]
        for j, (proj, d) in enumerate(cur):
            ev = events[j] if events is not None else None
            if ev is not None:
                ev[0].record()
            plans[j].fwd(d["X"], d["W"], d["A"], d["B"], proj.scale, d["Y"])
            if ev is None:       # the product path: lora_linear_bwd (dX GEMM beside the dA / dB passes where the plan says so)
                plans[j].bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"])
            else:                # the same kernels one after the other through the stage calls, with events between them
                plans[j].bwd_stages(d["dY"], d["X"], d["W"], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"], events=ev[1:])

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    n_warm = max(args.warmup, 3)
    for k in range(n_warm):
        step(k)
    torch.cuda.synchronize()
    for pl in plans:
        code, msg = pl.device_status()
        if code != 0:
            raise SystemExit(f"bench.py: device status after warm-up: {msg}")

    # ---- timed region: K steps back to back, device-timed (events only around the region) ----
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for k in range(n_warm):              # once more, so that the timed region starts from a loaded, warm GPU
        step(k)
    launches0 = binding.launch_count()
    barrier()
    torch.cuda.synchronize()
    t_host0 = time.time()
    ev_a.record()
    for k in range(args.steps):
        step(n_warm + k)
    ev_b.record()
    torch.cuda.synchronize()
    t_host1 = time.time()
    barrier()
    launches = binding.launch_count() - launches0
    ms_total = max_over_ranks(ev_a.elapsed_time(ev_b), device, world)
    ms_step = ms_total / args.steps

    # ---- the same steps once more with events between the kernels: per-kernel durations.  An event record between two
    #      launches suppresses their programmatic overlap, so this pass is a little slower than the timed region; its
    #      own per-step time is reported as ms_per_step_instrumented ----
    events = [[[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in protos] for _ in range(args.steps)]
    i_a, i_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    i_a.record()
    for k in range(args.steps):
        step(n_warm + k, events[k])
    i_b.record()
    torch.cuda.synchronize()
    t_host2 = time.time()
    ms_step_instr = i_a.elapsed_time(i_b) / args.steps
    clocks = sampler.stop(t_host0, t_host2) if sampler is not None else None

    # per-stage mean durations (ms) from the instrumented pass.  Events: 0 before the forward call, 1 after it, 2 after the
    # dY B pre-pass, 3 after the dX GEMM launch, 4 after the dA stage, 5 after the dB stage
    kern = {}
    for j, p in enumerate(protos):
        dur = [statistics.mean(events[k][j][i].elapsed_time(events[k][j][i + 1]) for k in range(args.steps)) for i in range(5)]
        fwd_flops = 2.0 * p.T * p.d_in * p.d_out + 2.0 * p.T * p.r * (p.d_in + p.d_out)
        dxg_flops = 2.0 * p.T * p.d_in * p.d_out + 2.0 * p.T * p.r * p.d_in            # dense + the rank-r k-block (Q A)
        q_bytes = 2.0 * p.T * p.d_out + 2.0 * p.T * p.r + 2.0 * p.r * p.d_out           # dY once, B in, Qt out
        da_bytes = 2.0 * p.T * p.d_in + 2.0 * p.T * p.r * 2 + 4.0 * p.r * p.d_in      # X once, Qt in, Pt out, dA out
        db_bytes = 2.0 * p.T * p.d_out + 2.0 * p.T * p.r + 4.0 * p.r * p.d_out        # dY once, Pt in, dB out
        kern[p.name] = {
            "fwd_stage": {"ms": dur[0], "tflops": fwd_flops / dur[0] / 1e9,
                          "frac_of_bf16_peak": fwd_flops / dur[0] / 1e9 / pk["bf16_tflops"]},
            "q_prepass": {"ms": dur[1], "gbs": q_bytes / dur[1] / 1e6, "frac_of_hbm_peak": q_bytes / dur[1] / 1e6 / pk["hbm_gbs"]},
            "dx_gemm": {"ms": dur[2], "tflops": dxg_flops / dur[2] / 1e9,
                        "frac_of_bf16_peak": dxg_flops / dur[2] / 1e9 / pk["bf16_tflops"]},
            "dA": {"ms": dur[3], "gbs": da_bytes / dur[3] / 1e6, "frac_of_hbm_peak": da_bytes / dur[3] / 1e6 / pk["hbm_gbs"]},
            "dB": {"ms": dur[4], "gbs": db_bytes / dur[4] / 1e6, "frac_of_hbm_peak": db_bytes / dur[4] / 1e6 / pk["hbm_gbs"]},
        }
    # dominant kernel for the roofline: the dX GEMM launch of the projection with the longest GEMMs.  Its event pair
    # brackets exactly ONE kernel (the K-extended CTA-pair GEMM; the dY B pre-pass sits before the first of the two events)
    # unless the plan splits it along K or the batch is too small for CTA pairs (then the bracket holds what dx_launches says)
    dom_p = max(protos, key=lambda p: kern[p.name]["fwd_stage"]["ms"] + kern[p.name]["dx_gemm"]["ms"])
    dom_plan = plans[protos.index(dom_p)].config()
    dom = kern[dom_p.name]["dx_gemm"]
    dx_launches = 1 + (1 if dom_plan["dx_split_k"] > 1 and dom_plan["cta_group"] == 2 else 0)
    roofline = {"bound": "tensor",
                "kernel": f"lora_gemm_pair_kernel<1,1>: dX = dY W + (s dY B) A as one K-extended GEMM ({dom_p.name})"
                          if dom_plan["cta_group"] == 2 else f"lora_gemm_kernel<1> (single-CTA dX GEMM, {dom_p.name})",
                "launches_in_bracket": dx_launches,
                "achieved": dom["tflops"], "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                "frac": dom["tflops"] / pk["bf16_tflops"], "peak_kind": f"bf16 burst, of {pk['source']}",
                "frac_of_sustained": dom["tflops"] / pk["bf16_tflops_sustained"],
                "ms_per_launch": dom["ms"],
                "flops_per_launch": 2.0 * dom_p.T * dom_p.d_in * dom_p.d_out + 2.0 * dom_p.T * dom_p.r * dom_p.d_in,
                "traffic": (NCU_TRAFFIC["bytes_per_launch"]["dx_gemm"] if NCU_TRAFFIC["gemm_sha"] == gemm_source_sha()
                            and args.workload == 1 else None)}

    # ---- variant: backward that reuses the forward's X A^T (lora_linear_bwd_saved_p), same inputs and rotation ----
    def step_saved(k):
        cur = sets[k % n_sets]
        for j, (proj, d) in enumerate(cur):
            plans[j].fwd(d["X"], d["W"], d["A"], d["B"], proj.scale, d["Y"])
            plans[j].bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"], saved_p=True)

    n_var = max(3, min(args.steps, 50))
    for k in range(3):
        step_saved(k)
    torch.cuda.synchronize()
    v_a, v_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    v_a.record()
    for k in range(n_var):
        step_saved(3 + k)
    v_b.record()
    torch.cuda.synchronize()
    barrier()
    ms_var = max_over_ranks(v_a.elapsed_time(v_b) / n_var, device, world)
    variants = {"bwd_saved_p": {"ms_per_step": ms_var, "value": job_value(world, flops_step, ms_var), "unit": UNIT,
                                "steps": n_var, "note": "forward + lora_linear_bwd_saved_p (X A^T kept from the forward)"}}

    # ---- variant: quantised LoRA (NF4 frozen weight): lora_linear_fwd_nf4 + lora_linear_bwd_nf4, same inputs.  Two forms:
    #      weight expanded once per call into a scratch buffer (fast), or expanded inside the GEMM kernels (no extra memory)
    if all(p.d_in % 64 == 0 for p in protos):
        q_sets = [[binding.nf4_quantize(d["W"]) for _, d in cur] for cur in sets]
        w_scratch = {}
        for p in protos:
            if (p.d_out, p.d_in) not in w_scratch:
                w_scratch[(p.d_out, p.d_in)] = torch.empty((p.d_out, p.d_in), dtype=torch.bfloat16, device=device)

        def step_nf4(k, scratch):
            cur, qs = sets[k % n_sets], q_sets[k % n_sets]
            for j, (proj, d) in enumerate(cur):
                ws = w_scratch[(proj.d_out, proj.d_in)] if scratch else None
                plans[j].fwd_nf4(d["X"], qs[j][0], qs[j][1], d["A"], d["B"], proj.scale, d["Y"], w_scratch=ws)
                plans[j].bwd_nf4(d["dY"], d["X"], qs[j][0], qs[j][1], d["A"], d["B"], proj.scale, d["dX"], d["dA"], d["dB"],
                                 w_scratch=ws)

        forms = [("q_lora_nf4", True, "weight expanded once per call into a bf16 scratch buffer, then the bf16 kernels")]
        if all(p.T > 128 for p in protos):
            forms.append(("q_lora_nf4_in_kernel", False, "no scratch: weight expanded inside the GEMM kernels, per 256-token tile"))
        for key, scratch, how in forms:
            for k in range(3):
                step_nf4(k, scratch)
            torch.cuda.synchronize()
            q_a, q_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            q_a.record()
            for k in range(n_var):
                step_nf4(3 + k, scratch)
            q_b.record()
            torch.cuda.synchronize()
            barrier()
            ms_q = max_over_ranks(q_a.elapsed_time(q_b) / n_var, device, world)
            variants[key] = {"ms_per_step": ms_q, "value": job_value(world, flops_step, ms_q), "unit": UNIT, "steps": n_var,
                             "tokens_per_s": world * tokens_step / ms_q * 1e3,
                             "note": "forward + backward with the frozen W in NF4 (4.5 bits per weight); " + how +
                                     "; same algorithmic FLOPs as the bf16 step"}
        del q_sets, w_scratch

    # ---- extra kernel: the dense weight gradient of full fine-tuning, dW = dY^T X (lora_dense_dw), per projection ----
    dw_out = [torch.empty((p.d_out, p.d_in), dtype=torch.bfloat16, device=device) for p in protos]

    def step_dw(k):
        cur = sets[k % n_sets]
        for j, (proj, d) in enumerate(cur):
            plans[j].dense_dw(d["dY"], d["X"], dw_out[j])

    for k in range(3):
        step_dw(k)
    torch.cuda.synchronize()
    w_a, w_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    w_a.record()
    for k in range(n_var):
        step_dw(3 + k)
    w_b.record()
    torch.cuda.synchronize()
    barrier()
    ms_dw = max_over_ranks(w_a.elapsed_time(w_b) / n_var, device, world)
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
    n_lanes = 1 if args.workload >= 4 else 2
    h_in = []
    for j, (p, d0) in enumerate(sets[0]):
        h_in.append({k: d0[k].cpu().pin_memory() for k in ("X", "A", "B", "dY")})
    lanes = []
    for ln in range(n_lanes):
        lp = plans if ln == 0 else [binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r, device=local_rank) for p in protos]
        for pl in lp:
            pl.ensure_workspace()
        outs = [{k: torch.empty_like(d0[k], device="cpu").pin_memory() for k in ("Y", "dX", "dA", "dB")} for _, d0 in sets[0]]
        stg = [torch.empty(lp[j].step_host_staging_bytes(), dtype=torch.uint8, device=device) for j in range(len(protos))]
        lanes.append({"plans": lp, "out": outs, "staging": stg, "stream": torch.cuda.Stream(device=device)})

    def step_host(k):
        ln = lanes[k % n_lanes]
        for j, (p, d0) in enumerate(sets[0]):
            h, ho = h_in[j], ln["out"][j]
            ln["plans"][j].step_host(h["X"], d0["W"], h["A"], h["B"], h["dY"], p.scale, ho["Y"], ho["dX"], ho["dA"], ho["dB"],
                                     ln["staging"][j], stream=ln["stream"])

    def run_host(n):
        cur = torch.cuda.current_stream()
        start, done = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(cur)
        for ln in lanes:
            ln["stream"].wait_event(start)
        for k in range(n):
            step_host(k)
        for ln in lanes:
            ev = torch.cuda.Event()
            ev.record(ln["stream"])
            cur.wait_event(ev)
        done.record(cur)
        torch.cuda.synchronize()
        return start.elapsed_time(done)

    n_e2e = max(4, min(args.steps, 20 if args.workload < 4 else 3))
    run_host(2 * n_lanes)
    barrier()
    ms_e2e = max_over_ranks(run_host(n_e2e) / n_e2e, device, world)
    barrier()
    h2d = sum(t.numel() * t.element_size() for h in h_in for t in h.values())
    d2h = sum(t.numel() * t.element_size() for ho in lanes[0]["out"] for t in ho.values())
    e2e = {"value": job_value(world, flops_step, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "ms_per_step": ms_e2e, "steps": n_e2e, "lanes": n_lanes,
           "pcie_gbs": {"h2d": h2d / ms_e2e / 1e6, "d2h": d2h / ms_e2e / 1e6},
           "note": "host X, A, B, dY in; Y, dX, dA, dB out (pinned); frozen W resident on the device; "
                   f"{n_lanes} lane(s) of lora_linear_step_host alternate so that copies of neighbouring steps overlap"}

    if rank != 0:
        return
    cpu = cpu_baseline(args.workload) if world == 1 and not args.no_cpu_baseline else None
    value = job_value(world, flops_step, ms_step)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": n_warm,
        "ms_per_step": ms_step, "ms_per_step_instrumented": ms_step_instr, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(args.workload), "projections": [p.name for p in protos], "T": protos[0].T,
                   "r": protos[0].r, "scale": protos[0].scale, "input_sets_rotated": n_sets, "grouped": bool(args.grouped and args.workload == 4),
                   "l2": f"{n_sets} independent input/output sets ({bytes_per_set * n_sets / 2**20:.0f} MiB) rotated per step; "
                         "each step's operands exceed the 126 MB L2",
                   "replicas": "independent replica per GPU, no collective"},
        "tokens_per_s": world * tokens_step / ms_step * 1e3,
        "frac_of_bf16_peak": value / world / pk["bf16_tflops"], "peak_source": pk["source"],
        "kernels": kern, "variants": variants, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        "plan": plans[0].describe(),
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--grouped", action="store_true",
                    help="workload 4 only: run q/k/v and gate/up as one grouped projection each (shared X)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

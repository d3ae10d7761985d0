"""Host-side logic of bench.py that needs no GPU: the multi-rank aggregation (two gloo ranks on CPU) and the
reference arm's rank handling."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    dist.barrier()
    slowest = bench.max_over_ranks(local_ms, torch.device("cpu"), world)
    value = bench.job_value(world, 2.0e12, slowest)    # each replica does 2 TFLOP per step
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"slowest": slowest, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_the_slowest_rank(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(2)]
    assert res[0] == res[1]
    assert res[0]["slowest"] == 15.0
    # 2 replicas x 2 TFLOP in 15 ms = 266.7 TFLOP/s for the job
    assert abs(res[0]["value"] - 2 * 2.0e12 / 15.0 / 1e9) < 1e-9


def test_single_rank_helpers():
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu"), 1) == 3.5
    assert bench.job_value(1, 556.2e9, 0.5) == 556.2e9 / 0.5 / 1e9
    assert bench.workload_name(1).startswith("config1 q_proj")
    pk = bench.peaks()
    assert pk["hbm_gbs"] > 1000 and pk["bf16_tflops"] > 500 and pk["source"] in ("measured", "fallback")
    assert len(bench.source_sha("gemm")) == 16 and bench.source_sha("gemm") != bench.source_sha("adapter_grad")
    p = bench.inputs_workload(1)[0]
    assert bench.stage_bytes(p, "grads") > bench.stage_bytes(p, "dA") + bench.stage_bytes(p, "dB") - 4.0 * p.T * p.r - 1


def test_reference_arm_prints_one_line_on_rank0_and_nothing_elsewhere():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "0"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["dtype"] == "f64" and line["gpu_launches"] == 0

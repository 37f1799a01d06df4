"""bench.py end to end on small workloads: the one-GPU record with its checks, and the partitioned arm (the code
path of N > 1) on a single rank with NCCL."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, cwd=ROOT, timeout=900)
    assert r.returncode == 0, (r.stdout[-2000:], r.stderr[-2000:])
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_single_gpu_record_carries_its_checks():
    d = run_bench("--workload", "medium", "--scale", "0.02", "--steps", "3", "--warmup", "3", "--cpu-seconds", "1")
    assert d["n_gpus"] == 1 and d["value"] > 0 and d["rejected"] is False and d["problems"] == []
    assert d["config"]["workload"].startswith("medium") and d["dtype"] == "f32"
    assert d["parity"]["ok"] and d["parity"]["stored"]["max_rel"] <= 1e-4 and d["parity"]["exact"]["max_rel"] <= 1e-4
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0 and d["e2e"]["buffer_sets"] == 2
    assert d["roofline"]["bound"] == "hbm" and d["roofline"]["achieved"] > 0 and d["gpu_launches"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["result_check"]["finite"]
    assert abs(d["instrumented_ms_per_step"] - d["ms_per_step"]) < 0.25 * d["ms_per_step"]


@pytest.mark.parametrize("layout", ["gather", "partial"])
def test_partitioned_arm_on_one_rank(layout):
    d = run_bench("--workload", "medium", "--scale", "0.02", "--steps", "2", "--warmup", "3", "--layout", layout)
    assert d["scaling"] == "strong" and d["n_gpus"] == 1 and d["value"] > 0 and d["rejected"] is False
    assert "vertex ranges" in d["config"]["parallelism"] and d["result_check"]["finite"]
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["gpu_launches"] > 0


def test_tiny_latency_record_and_cuda_graph_replay():
    """The Tiny workload as the benchmark reports it: latency of one it_infer, call by call and replayed from a CUDA
    graph captured around the same call (the library allocates nothing and synchronises nothing inside it_infer)."""
    import sys
    sys.path.insert(0, ROOT)
    import torch
    import bench
    rec = bench.measure_tiny(None, torch.device("cuda"))
    assert rec["parity"]["ok"] and rec["problems"] == []
    assert rec["us_per_infer"] > 0 and rec["launches_per_infer"] > 0
    assert rec.get("cuda_graph_error") is None, rec.get("cuda_graph_error")
    assert rec["cuda_graph_result_identical"] and rec["us_per_infer_cuda_graph"] > 0


def test_headline_workload_at_a_small_size_runs_the_fused_pair_and_the_unsplit_pass():
    """The bf16 model of the headline workload: its two dense products around the layer boundary run as one kernel
    (gemm2_tc in the kernel list, no gemm_tc), the sampled parity holds, and the pass without the vertex split is
    timed beside it (the threshold is lowered so that this small graph has hubs to split)."""
    d = run_bench("--workload", "large", "--scale", "0.002", "--threshold", "256", "--steps", "3", "--warmup", "3",
                  "--cpu-seconds", "1", "--no-others")
    assert d["rejected"] is False and d["problems"] == [] and d["dtype"] == "bf16"
    names = {k["name"] for k in d["kernels"]}
    assert "gemm2_tc" in names and "gemm_tc" not in names
    assert d["parity"]["ok"] and d["parity"]["stored"]["max_rel"] <= 2e-2
    assert d["split"]["split_owners"] > 0 and d["unsplit"]["ms_per_step"] > 0 and d["unsplit"]["value"] > 0

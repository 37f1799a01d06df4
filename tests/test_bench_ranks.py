"""The multi-rank side of bench.py on CPU: world_size-2 gloo ranks.

With N > 1 the benchmark partitions one workload over the ranks (tests/test_sharded_cpu.py covers the partition and
the exchanges); what is checked here is the timing protocol the ranks share (the slowest rank's time, the whole-job
value) and the rule that rank 0 alone reports.
"""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 * (rank + 1)            # rank 0: 10 ms, rank 1: 20 ms
    ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    value = bench.whole_job_value(1000, world, ms)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"ms": ms, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_slowest_rank_sets_the_whole_job_value(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for g in got:
        assert g["ms"] == 20.0                       # max over ranks, on every rank
        assert g["value"] == 2 * 1000 / 20e-3        # units of all ranks / the slowest rank's time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu")) == 7.5
    assert bench.whole_job_value(10, 1, 5.0) == 2000.0


def test_reference_arm_under_two_ranks_prints_one_line():
    """Launched the way the driver launches N > 1: rank 0 alone times the oracle and prints, the others exit 0."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--workload", "tiny", "--steps", "1", "--warmup", "0", "--cpu-seconds", "1"]
    r = subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_reference_arm_prints_one_contract_line():
    """`bench.py --impl reference` times the CPU oracle on a bounded sample and prints one JSON line with the
    keys the benchmark contract names (also with edge features in the messages)."""
    for extra in ([], ["--edge-dim", "8"]):
        out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                              "--steps", "2", "--warmup", "1", "--cpu-seconds", "1"] + extra,
                             capture_output=True, text=True, check=True, cwd=ROOT).stdout.strip().splitlines()
        assert len(out) == 1
        d = json.loads(out[0])
        assert d["impl"] == "reference" and d["unit"] == "vertices/s" and d["higher_is_better"] is True
        assert d["steps"] == 2 and d["warmup"] == 1 and d["n_gpus"] == 1 and d["value"] > 0 and d["dtype"] == "f64"
        assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
        assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
        assert d["config"]["workload"] == "tiny" and d["config"]["edge_feature_dim"] == (8 if extra else 0)

"""Multi-rank plumbing of bench.py on CPU: two gloo ranks combine their timings the way the
benchmark does (slowest rank's time, sum of units); the reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["CR_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
elapsed, units = bench.combine_ranks(1.0 + rank, 10.0 * (rank + 1), dist.get_world_size(), dist, None)
print(json.dumps({"rank": rank, "elapsed": elapsed, "units": units}))
dist.destroy_process_group()
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_report_slowest_time_and_total_units():
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CR_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["elapsed"] == 2.0 and o["units"] == 30.0


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.combine_ranks(0.5, 7.0, 1) == (0.5, 7.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line():
    env = dict(os.environ)
    env.pop("RANK", None)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1", "--ref-columns", "4096", "--workload", "cfg2"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("cfg2")


def test_reference_arm_of_a_regression_workload():
    """Regression workloads time the oracle's gradient-descent step (gradients of a sample of the
    partitions, aggregation of all, model update); other ranks print nothing."""
    env = dict(os.environ)
    env.pop("RANK", None)
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "3", "--warmup", "1",
           "--workload", "cfg1"]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and "partitions per step" in line["cpu_baseline"]["sample"]
    assert line["config"]["workload"].startswith("cfg1") and line["dtype"] == "f64"
    quiet = subprocess.run(cmd, env=dict(env, RANK="1", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    assert quiet.returncode == 0 and quiet.stdout.strip() == ""


def test_tree_override_keeps_the_partition_count_feasible():
    """`--tree n,L,s,code[,c]` sets P to c times the smallest count the tree can split into whole chunks:
    the oracle's allocation accepts it and gives every node c (s+1)^L slots."""
    sys.path.insert(0, ROOT)
    import bench
    from oracle import cr_oracle as O
    from oracle import cr_setup
    for text, c in (("12,1,1,cyclic", 1), ("4,3,1,cyclic,2", 2), ("6,2,2,repetition", 1)):
        cfg = bench.apply_tree_override(dict(d=64, seed=0), text)
        n, L, s = cfg["n"], cfg["L"], cfg["s"]
        assert cfg["P"] == c * O.partition_quantum(n, L, s)
        _, local, _ = cr_setup.setup(cfg)
        assert len(local) == O.num_nodes(n, L) and all(len(pairs) == c * (s + 1) ** L for pairs in local)

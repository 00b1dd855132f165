"""CPU-side checks of bench.py: the reference arm (the oracle timed on host cores) prints the contract's JSON
line, and the multi-rank aggregation (max of per-rank times over torch.distributed) works with two gloo ranks."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "agent-steps/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("cfg1_") and line["higher_is_better"] is True
    for key in ("metric", "n_gpus", "steps", "warmup", "ms_per_step", "scaling", "vs_baseline", "dtype", "data"):
        assert key in line


def _rank_main(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    r, w, _ = bench.dist_setup(world)
    assert (r, w) == (rank, world)
    bench.dist_barrier(w)
    got = bench.dist_max(10.0 + rank, w, device="cpu")    # every rank must see the slowest rank's time
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(str(got))
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_rank_time_aggregation_gloo(tmp_path):
    mp.spawn(_rank_main, args=(2, 29533, str(tmp_path)), nprocs=2, join=True)
    assert [float(open(tmp_path / f"r{k}.txt").read()) for k in range(2)] == [11.0, 11.0]


def test_algorithmic_bytes_formula():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2205_05248_b200 import workloads
    cfg = workloads.config(5)
    assert abs(bench.algorithmic_bytes_per_agent_step(cfg, 64) - 737.25) < 1e-9
    assert abs(bench.flops_per_agent_step(cfg) - (2 * 64 * (80 + 384 + 14) + 25 * 64)) < 1e-9

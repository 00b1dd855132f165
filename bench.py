#!/usr/bin/env python
"""Benchmark of the batched actor path: agent-steps per second on one B200, ring write included.

One bench "step" is one ``marl_rollout_staged`` call: T environment steps over all E environments, i.e. one
pass of the whole hot path (stage obs, network, choice, ring write, episode bookkeeping) over one batch of
synthetic environment output that is already resident in HBM (generated once, before the timed region,
by ``marl_env_generate``).  The default workload is the largest one of the throughput sweep
(E=65536 x 8 agents, obs 80, 14 actions, hidden 64, bf16, T=64, ring of about 20 GB).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 5 --E 65536 --H 64 --precision bf16]
                    [--kernel auto|ffma|tensor] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torchrun, one rank per GPU) every rank runs its own
replica of the workload - environments are independent, there is no data-path collective - and the value
is the sum over ranks divided by the slowest rank's time ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
METRIC = "agent-steps/sec at 1 B200 (incl. ring write); % of step roofline (HBM/TC)"
UNIT = "agent-steps/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=5)
    ap.add_argument("--E", type=int, default=None)
    ap.add_argument("--H", type=int, default=None)
    ap.add_argument("--precision", default=None, choices=[None, "fp32", "bf16"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "ffma", "tensor", "pipelined", "dual"])
    ap.add_argument("--refresh", action="store_true",
                    help="publish a new network during every step, effective at the middle of the next rollout "
                         "(the learner's model update running beside the workers)")
    ap.add_argument("--subset", type=float, default=0.0, metavar="FRACTION",
                    help="time marl_actor_step_subset instead: every call steps a seeded list of FRACTION * E "
                         "environments (a multiple of four), T calls per step")
    ap.add_argument("--lagged", action="store_true",
                    help="with --subset: marl_actor_step_lagged (reward/done are the outcome of the previous action)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--crossover", action="store_true",
                    help="time the CUDA-core, one-tile and pipelined kernels on the same bf16 rollouts over a range of "
                         "batch sizes (E x n rows from 24 to 16384): the evidence behind the automatic kernel choice")
    ap.add_argument("--sampler", type=int, default=0, metavar="B",
                    help="measure the learner-side episode sampler instead: draws of B episodes from a filled ring")
    return ap.parse_args()


def algorithmic_bytes_per_agent_step(cfg: dict, T: int) -> float:
    """Bytes that one agent-step of a tile-major rollout must move to and from HBM:
    reads  obs 4D + avail A + (reward 4 + done 1)/n, writes the ring record's payload
    obs 4D + avail A + action 4 + Q 4A + (reward 4 + done 1)/n, plus the hidden state loaded and stored once
    per launch (8H/T).  Padding, headers and weights are not counted."""
    D, A, n, H = cfg["D"], cfg["A"], cfg["n"], cfg["H"]
    reads = 4 * D + A + 5.0 / n
    writes = 4 * D + A + 4 + 4 * A + 5.0 / n
    return reads + writes + 8.0 * H / T


def flops_per_agent_step(cfg: dict) -> float:
    D, A, H = cfg["D"], cfg["A"], cfg["H"]
    return 2.0 * H * (D + 6 * H + A) + 25.0 * H


def traffic_record(kernel_name: str, agent_steps_per_launch: float, algorithmic_bytes: float) -> dict:
    """DRAM bytes per launch from the committed ncu record of this kernel: {"traffic": bytes or None, ...}.  None if
    there is no record or the kernel sources have changed since the counters were taken.  The record comes from a
    small case and is scaled by the agent-steps of a launch; where the scaled figure falls below the algorithmic
    bytes (the small case ends with part of its last writes still in L2), it is a lower bound and says so."""
    import hashlib
    path = os.path.join(ROOT, "profiles", f"{kernel_name}_traffic.txt")
    if not os.path.exists(path):
        return {"traffic": None}
    rec = {}
    for line in open(path):
        if line.startswith("#") or ":" not in line:
            continue
        k, v = line.split(":", 1)
        rec[k.strip()] = v.strip()
    try:
        h = hashlib.sha256()
        for f in rec["source_files"].split():
            h.update(open(os.path.join(ROOT, f), "rb").read())
        if h.hexdigest() != rec["source_sha256"]:
            return {"traffic": None}
        scaled = float(rec["dram_bytes_per_agent_step"]) * agent_steps_per_launch
    except (KeyError, OSError, ValueError):
        return {"traffic": None}
    note = (f"ncu capture of {rec.get('capture_agent_steps', '?')} agent-steps scaled to one launch"
            + ("; below the algorithmic bytes: a lower bound (the small case ends with writes still in L2)"
               if scaled < algorithmic_bytes else ""))
    return {"traffic": scaled, "traffic_note": note}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [x.strip() for x in line.split(",")]))

    def stop(self, t_begin: float, t_end: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [r for (ts, r) in self.rows if t_begin <= ts <= t_end + 0.05] or [r for (_, r) in self.rows]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_setup(n_gpus: int):
    """Returns (rank, world, local_rank).  torch.distributed is used only for the barrier and the max of the
    per-rank times; the data path has no collective."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch
        import torch.distributed as dist
        if torch.cuda.is_available():
            torch.cuda.set_device(local)
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
    return rank, world, local


def dist_max(value: float, world: int, device="cuda") -> float:
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def dist_barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def cpu_baseline(cfg: dict, weights: dict, budget_s: float = 15.0) -> dict:
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the workload."""
    import numpy as np
    import oracle
    cores = oracle.hardware_threads()
    T = cfg["T"]
    probe = min(cfg["E"], max(cores, 8))
    sess = oracle.Session(cfg, weights, np.arange(probe), with_ring=True, n_threads=cores)
    t0 = time.perf_counter()
    sess.rollout(cfg["env"], min(T, 8), cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"], trace=())
    dt = time.perf_counter() - t0
    rate = probe * cfg["n"] * min(T, 8) / dt
    envs = int(min(cfg["E"], max(probe, rate * budget_s / (cfg["n"] * T))))
    sess = oracle.Session(cfg, weights, np.arange(envs), with_ring=True, n_threads=cores)
    t0 = time.perf_counter()
    sess.rollout(cfg["env"], T, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"], trace=())
    dt = time.perf_counter() - t0
    return {"value": envs * cfg["n"] * T / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {envs} of {cfg['E']} environments x T={T} steps, {dt:.1f} s"}


def run_reference(args, cfg, rank):
    """--impl reference: the CPU oracle on the host cores, same metric and workload, bounded sample per step."""
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2205_05248_b200 import workloads
    weights = workloads.make_weights(cfg)
    cores = oracle.hardware_threads()
    T = cfg["T"]
    envs = min(cfg["E"], 4 * cores)
    times = []
    for k in range(args.warmup + args.steps):
        sess = oracle.Session(cfg, weights, np.arange(envs), with_ring=True, n_threads=cores)
        t0 = time.perf_counter()
        sess.rollout(cfg["env"], T, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"], trace=())
        dt = time.perf_counter() - t0
        if k >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = envs * cfg["n"] * T * len(times) / total
    sample = f"first {envs} of {cfg['E']} environments x T={T} steps per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg["name"], "step": f"one rollout of T={T} steps", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_sampler(args, cfg, dev):
    """--sampler B: fills the ring with a rollout long enough to close episodes everywhere, then times draws of B
    episodes (marl_ring_sample) with CUDA events.  Algorithmic bytes: every sampled record read once, every element
    of the dense batch written once."""
    import torch
    from paper_2205_05248_b200 import binding, workloads
    cfg = dict(cfg, env=dict(cfg["env"], done_thresh24=int(0.05 * (1 << 24))))   # episodes of about 20 steps
    weights = workloads.make_weights(cfg)
    actor = binding.Actor(cfg, device=str(dev), kernel=args.kernel, work_steps=8)
    actor.set_weights(weights)
    actor.rollout(cfg["env"], max(cfg["T"], 64), cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    B, L, n, D, A = args.sampler, cfg["L"], cfg["n"], cfg["D"], cfg["A"]
    out = None
    for k in range(args.warmup):
        out = actor.ring_sample(k, B)
    torch.cuda.synchronize()
    lens = out["len"].double()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for k in range(args.steps):
        actor.ring_sample(1000 + k, B)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / args.steps
    payload = 4 * n * D + n * A + 4 * n + 4 * n * A + 5                     # bytes of one step's fields
    bytes_per_draw = float(lens.sum()) * payload + B * L * payload + B * 16
    peaks, peak_kind = load_peaks()
    achieved = bytes_per_draw / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "episodes/s gathered by marl_ring_sample", "value": B / (ms * 1e-3), "unit": "episodes/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "u8", "data": "synthetic",
                      "config": {"workload": cfg["name"], "B": B, "L": L, "mean_len": float(lens.mean()),
                                 "complete_fraction": float((out["slot"] >= 0).double().mean())},
                      "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": peak_kind,
                                   "kernel": "ring_gather_kernel"}}), flush=True)
    actor.destroy()


def run_crossover(args, dev):
    """--crossover: one rollout of T=32 steps per launch, bf16, on the 3-agent and the 8-agent shapes, for every
    kernel that takes the shape, over batch sizes from one partial tile to many waves.  Each launch is timed with
    its own event pair; the median of the repetitions is reported in microseconds per environment step.  (The
    3-agent, 30-feature shape of the smallest experiment is taken by the CUDA-core kernel only.)"""
    import torch
    from paper_2205_05248_b200 import binding, workloads
    T, reps = 32, max(10, args.steps)
    rows_list = [24, 48, 96, 192, 384, 768, 1536, 3072, 6144, 16384]
    table = []
    for shape in (dict(n=3, D=30, A=9), dict(n=4, D=32, A=8), dict(n=8, D=80, A=14), dict(n=5, D=80, A=11)):
        for rows in rows_list:
            E = max(1, rows // shape["n"])
            cfg = workloads.small_config(H=64, precision="bf16", E=E, C=E, L=64, T=T, **shape)
            weights = workloads.make_weights(cfg)
            entry = {"n": shape["n"], "D": shape["D"], "A": shape["A"], "E": E, "rows": E * shape["n"]}
            for kernel in ("ffma", "tensor", "pipelined"):
                try:
                    actor = binding.Actor(cfg, device=str(dev), kernel=kernel, work_steps=1)
                except binding.MarlError:
                    entry[kernel] = None          # the kernel does not take this shape
                    continue
                actor.set_weights(weights)
                staged = actor.env_generate(cfg["env"], 0, T)
                for _ in range(3):
                    actor.rollout_staged(*staged, T, 0.05)
                torch.cuda.synchronize()
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
                ev[0].record()
                for k in range(reps):
                    actor.rollout_staged(*staged, T, 0.05)
                    ev[k + 1].record()
                torch.cuda.synchronize()
                assert actor.status()[0] == 0
                per = sorted(ev[k].elapsed_time(ev[k + 1]) for k in range(reps))
                entry[kernel] = round(1e3 * per[len(per) // 2] / T, 3)
                actor.destroy()
                del staged
            table.append(entry)
    print(json.dumps({"metric": "microseconds per environment step (median launch of T=32 steps), by kernel and batch",
                      "unit": "us/step", "higher_is_better": False, "dtype": "bf16", "data": "synthetic", "steps": reps,
                      "table": table}), flush=True)


def run_subset(args, cfg, dev):
    """--subset FRACTION: T calls of marl_actor_step_subset per step, each over one of four seeded lists of
    M = FRACTION * E environments in random order, the dense inputs of each list resident in HBM beforehand.
    Algorithmic bytes per agent-step: the one-step figure (hidden state loaded and stored by every call) plus the
    list entry."""
    import numpy as np
    import torch
    from paper_2205_05248_b200 import binding, workloads
    T, E, n = cfg["T"], cfg["E"], cfg["n"]
    M = max(4, int(args.subset * E) // 4 * 4)
    weights = workloads.make_weights(cfg)
    actor = binding.Actor(cfg, device=str(dev), kernel=args.kernel, work_steps=1)
    actor.set_weights(weights)
    staged = actor.env_generate(cfg["env"], 0, 4)
    rng = np.random.default_rng(cfg["seed"])
    lists = [rng.permutation(E)[:M].astype(np.int32) for _ in range(4)]
    inputs = []
    for k, ids in enumerate(lists):
        tid = torch.as_tensor(ids, device=dev, dtype=torch.long)
        inputs.append([t[k].index_select(0, tid).contiguous() for t in staged])
    acts = torch.empty((M, n), dtype=torch.int32, device=dev)
    del staged

    step = actor.step_lagged if args.lagged else actor.step_subset

    def one_step():
        for k in range(T):
            step(lists[k % 4], *inputs[k % 4], cfg["eps_start"], acts)

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    launches0 = actor.launch_count
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        one_step()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    launches = actor.launch_count - launches0
    status, _ = actor.status()
    assert status == 0, f"device status {status}"
    per_step = algorithmic_bytes_per_agent_step(cfg, 1) + 4.0 / n
    kernel_ms = ms / launches
    achieved = per_step * M * n / (kernel_ms * 1e-3) / 1e9
    peaks, peak_kind = load_peaks()
    in_bytes = sum(t.numel() * t.element_size() for t in inputs[0])
    print(json.dumps({"metric": METRIC, "value": M * n * T * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
                      "higher_is_better": True, "dtype": cfg["precision"], "data": "synthetic",
                      "config": {"workload": cfg["name"], "E": E, "M": M, "n": n, "T": T, "kernel": actor.kernel_name,
                                 "step": f"T={T} {'marl_actor_step_lagged' if args.lagged else 'marl_actor_step_subset'} calls over lists of M={M} of E={E} environments",
                                 "l2": f"each call reads {in_bytes / 1e6:.0f} MB of inputs and {M * n * cfg['H'] * 4 / 1e6:.0f} MB of "
                                       "hidden state (four lists in turn)"},
                      "gpu_launches": int(launches),
                      "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": peak_kind,
                                   "kernel_ms": kernel_ms, "algorithmic_bytes_per_agent_step": per_step}}), flush=True)
    actor.destroy()


def main():
    args = parse_args()
    from paper_2205_05248_b200 import workloads
    cfg = workloads.config(args.workload, E=args.E, H=args.H, precision=args.precision)
    rank, world, local = dist_setup(args.gpus)
    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return
    if args.warmup < 3:
        args.warmup = 3

    import torch
    from paper_2205_05248_b200 import binding
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if args.sampler > 0:
        if rank == 0:
            run_sampler(args, cfg, dev)
        return
    if args.crossover:
        if rank == 0:
            run_crossover(args, dev)
        return
    if args.subset > 0:
        if rank == 0:
            run_subset(args, cfg, dev)
        return
    cfg["seed"] = cfg["seed"] + (rank << 20)          # every rank runs its own replica
    cfg["env"] = dict(cfg["env"], seed=cfg["env"]["seed"] + (rank << 20))
    T, E, n = cfg["T"], cfg["E"], cfg["n"]
    weights = workloads.make_weights(cfg)

    actor = binding.Actor(cfg, device=str(dev), kernel=args.kernel, work_steps=1)
    actor.set_weights(weights)
    staged = actor.env_generate(cfg["env"], 0, T)      # resident in HBM before the timed region
    input_bytes = sum(t.numel() * t.element_size() for t in staged)
    torch.cuda.synchronize()

    nets = [weights, workloads.make_weights(cfg, seed=cfg["seed"] + 1)]
    done_steps = [0]

    def one_step():
        if args.refresh:
            k = done_steps[0] // T + 1
            actor.publish_weights(nets[k % 2], version=k + 1, effective_step=done_steps[0] + T // 2)
        actor.rollout_staged(*staged, T, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
        done_steps[0] += T

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    sampler.start()
    time.sleep(0.25)
    launches0 = actor.launch_count
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]   # one pair per step
    dist_barrier(world)
    torch.cuda.synchronize()
    t_begin = time.perf_counter()
    evs[0].record()
    for k in range(args.steps):
        one_step()
        evs[k + 1].record()
    torch.cuda.synchronize()
    t_end = time.perf_counter()
    dist_barrier(world)
    clocks = sampler.stop(t_begin, t_end)
    launches = actor.launch_count - launches0
    ms_local = evs[0].elapsed_time(evs[-1])
    ms_median = statistics.median(evs[k].elapsed_time(evs[k + 1]) for k in range(args.steps))
    ms_total = dist_max(ms_local, world)
    status, counters = actor.status()
    assert status == 0, f"device status {status}"
    agent_steps = E * n * T * args.steps
    value = world * agent_steps / (ms_total * 1e-3)

    peaks, peak_kind = load_peaks()
    kernel_ms = ms_local / max(launches, 1)            # one actor kernel per bench step (two when it is split)
    T_launch = T * args.steps / max(launches, 1)       # environment steps one launch covers
    bytes_per_launch = algorithmic_bytes_per_agent_step(cfg, T_launch) * E * n * T_launch
    achieved = bytes_per_launch / (kernel_ms * 1e-3) / 1e9
    flop_rate = flops_per_agent_step(cfg) * E * n * T_launch / (kernel_ms * 1e-3) / 1e12
    kname = {"tcgen05-pipelined": "actor_tcp_kernel", "tcgen05": "actor_tc_kernel", "tcgen05-dual": "actor_tc2_kernel",
             "tcgen05-streamed": "actor_tcw_kernel"}.get(actor.kernel_name, "actor_ffma_kernel")
    if cfg["precision"] == "fp32":
        # the fp32 path is bound by plain FFMA arithmetic: peak measured on this device by the library's FMA loop
        ffma_peak = binding.marl_measure_ffma_tflops()
        roofline = {"bound": "alu", "achieved": flop_rate, "peak": ffma_peak, "unit": "TFLOP/s",
                    "frac": flop_rate / ffma_peak, "traffic": None, "peak_source": "measured (FFMA loop, this run)",
                    "kernel": kname, "kernel_ms": kernel_ms, "flops_per_agent_step": flops_per_agent_step(cfg),
                    "hbm_gbs_achieved": achieved}
    else:
        # The step's roofline is the slower of its bytes at the measured HBM bandwidth and its FLOPs at the measured
        # bf16 tensor throughput (the sustained figure: the timed region is a loop of seconds).
        tf_peak = peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"]
        t_hbm = bytes_per_launch / (peaks["hbm_gbs"] * 1e9)
        t_tensor = flops_per_agent_step(cfg) * E * n * T_launch / (tf_peak * 1e12)
        common = {"peak_source": peak_kind, "kernel": kname, "kernel_ms": kernel_ms,
                  "algorithmic_bytes_per_agent_step": algorithmic_bytes_per_agent_step(cfg, T_launch),
                  "flops_per_agent_step": flops_per_agent_step(cfg), "hbm_gbs_achieved": achieved,
                  "tflops_effective": flop_rate, "hbm_frac": achieved / peaks["hbm_gbs"], "tensor_frac": flop_rate / tf_peak}
        if t_tensor > t_hbm:
            roofline = {"bound": "tensor", "achieved": flop_rate, "peak": tf_peak, "unit": "TFLOP/s",
                        "frac": flop_rate / tf_peak, "traffic": None, **common}
        else:
            roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": achieved / peaks["hbm_gbs"], **traffic_record(kname, E * n * T_launch, bytes_per_launch),
                        **common}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "ms_per_step_median": ms_median,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg["precision"], "data": "synthetic",
            "config": {"workload": cfg["name"], "E": E, "n": n, "D": cfg["D"], "A": cfg["A"], "H": cfg["H"], "T": T,
                       "ring": f"{cfg['C']}x{cfg['L']}", "kernel": actor.kernel_name,
                       "step": f"one marl_rollout_staged call = T={T} environment steps over E={E} environments",
                       "l2": f"inputs larger than L2 ({input_bytes / 1e6:.0f} MB staged per step, read once)"},
            "clocks": clocks, "gpu_launches": int(launches), "roofline": roofline}
    if args.refresh:
        line["config"]["weight_refresh"] = (f"one publication per step, effective {T // 2} environment steps into the "
                                            f"rollout (the launch is split there); final version {actor.weights_version}")

    # ---- end to end through the host-buffer entry point: H2D of each step's inputs, D2H of its actions ----
    if not args.no_e2e:
        distinct = min(T, 4)
        host = [[t[k].cpu().pin_memory() for t in staged] for k in range(distinct)]
        h_act = torch.empty((E, n), dtype=torch.int32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in host[0]) * T
        d2h = h_act.numel() * 4 * T
        e2e_steps = max(1, min(args.steps, 5))
        for k in range(2):
            actor.step_host(*host[k % distinct], cfg["eps_start"], h_act)
        dist_barrier(world)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            for k in range(T):
                actor.step_host(*host[k % distinct], cfg["eps_start"], h_act)
        torch.cuda.synchronize()
        dt = dist_max(time.perf_counter() - t0, world)
        line["e2e"] = {"value": world * E * n * T * e2e_steps / dt, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                       "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                       "call": "marl_actor_step_host x T per step (pinned host buffers, actions read back)"}
        del host

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        actor.destroy()
        del staged
        line["cpu_baseline"] = cpu_baseline(cfg, weights)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

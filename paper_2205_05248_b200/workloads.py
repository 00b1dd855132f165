"""Seeded synthetic workloads: the shapes of the experiments and the network weights.

This module holds *inputs only* - dimensions, probabilities turned into integer thresholds, and the
weight tensors drawn from a seeded generator.  It contains none of the actor step's arithmetic and is
the one module that both the CUDA library's callers and the CPU oracle's callers may import; the same
arrays are handed to both sides.

Shapes (agents, actions, observation width) are those of the four scenarios in Table II of the paper;
the simulator itself is replaced by a seeded synthetic environment described by ``env`` below.
"""
from __future__ import annotations

import math

import numpy as np

SEED_BASE = 0x5EED0000


def thresh24(p: float) -> int:
    """Probability -> 24-bit integer threshold: event iff (word >> 8) < floor(p * 2^24)."""
    return int(math.floor(p * (1 << 24)))


def _env(seed, obs_law, p_done, p_first, p_rest, split, n_type0=0, tb_start=0, tb_len=0):
    return dict(seed=seed, obs_law=obs_law, done_thresh24=thresh24(p_done),
                avail_thresh_first=thresh24(p_first), avail_thresh_rest=thresh24(p_rest), avail_split=split,
                n_type0=n_type0, type_block_start=tb_start, type_block_len=tb_len,
                p_done=p_done, p_first=p_first, p_rest=p_rest)


def config(k: int, E: int | None = None, H: int | None = None, precision: str | None = None) -> dict:
    """The k-th workload (1..5).  Workload 5 is a sweep: E in {4096,16384,65536}, H in {64,128}, both
    precisions; its defaults are the largest E, H=64, bf16.

    Returns a dict with the actor dimensions (E n D A H C L precision seed), the rollout parameters
    (T eps_start eps_end anneal_steps) and the synthetic-environment description ``env``.
    """
    seed = SEED_BASE + k
    if k == 1:    # 3 agents, 9 actions, obs 30 (scenario "3m")
        c = dict(E=8, n=3, D=30, A=9, H=64, C=64, L=32, precision="fp32", T=16, eps_start=0.05, eps_end=0.05,
                 anneal_steps=0, env=_env(seed, 0, 0.02, 0.8, 0.8, 9))
    elif k == 2:  # 8 agents, 14 actions, obs 80 ("8m")
        c = dict(E=1024, n=8, D=80, A=14, H=64, C=2048, L=128, precision="bf16", T=128, eps_start=0.1,
                 eps_end=0.1, anneal_steps=0, env=_env(seed, 1, 0.008, 0.7, 0.7, 14))
    elif k == 3:  # 5 agents of two unit types, 11 actions, obs 80 ("2s3z")
        c = dict(E=4096, n=5, D=80, A=11, H=64, C=8192, L=256, precision="bf16", T=256, eps_start=1.0,
                 eps_end=0.05, anneal_steps=255, env=_env(seed, 0, 0.006, 0.75, 0.75, 11, 2, 48, 16))
    elif k == 4:  # 5 agents, 12 actions of which the last 6 are attack targets, obs 55 ("5m_vs_6m")
        c = dict(E=16384, n=5, D=55, A=12, H=64, C=16384, L=128, precision="bf16", T=128, eps_start=0.05,
                 eps_end=0.05, anneal_steps=0, env=_env(seed, 0, 0.01, 0.9, 0.5, 6))
    elif k == 5:  # throughput sweep on the "8m" shape; ring of about 20 GB
        E = 65536 if E is None else E
        H = 64 if H is None else H
        idx = {4096: 0, 16384: 1, 65536: 2}.get(E, 3) * 2 + (0 if H == 64 else 1)
        seed = SEED_BASE + 5 + 16 * (idx + 1)
        c = dict(E=E, n=8, D=80, A=14, H=H, C=max(65536, E), L=96, precision="bf16", T=64, eps_start=0.05,
                 eps_end=0.05, anneal_steps=0, env=_env(seed, 0, 0.005, 0.7, 0.7, 14))
    else:
        raise ValueError("workload index must be 1..5")
    if E is not None and k != 5:
        assert c["C"] % c["E"] == 0
        S = c["C"] // c["E"]
        c["E"] = E
        c["C"] = E * S
    if H is not None:
        c["H"] = H
    if precision is not None:
        c["precision"] = precision
    c["seed"] = seed
    c["name"] = f"cfg{k}_E{c['E']}_n{c['n']}_D{c['D']}_A{c['A']}_H{c['H']}_{c['precision']}"
    return c


def small_config(**over) -> dict:
    """A tiny workload for unit tests; any key can be overridden."""
    c = dict(E=4, n=3, D=6, A=5, H=8, C=8, L=6, precision="fp32", T=8, eps_start=0.2, eps_end=0.2,
             anneal_steps=0, seed=SEED_BASE + 99, name="small")
    c.update({k: v for k, v in over.items() if k != "env"})
    env = _env(c["seed"], 0, 0.15, 0.7, 0.7, c["A"])
    env.update(over.get("env", {}))
    c["env"] = env
    return c


def make_weights(cfg: dict, seed: int | None = None, bias_scale: float = 1.0) -> dict:
    """Network weights as float32 arrays in [out][in] layout.

    Matrices: Xavier-uniform U(-a, a) with a = sqrt(6 / (fan_in + fan_out)).  Biases: U(-b, b) with
    b = bias_scale / sqrt(fan_in) (non-zero so that a dropped bias shows up in a comparison).
    W_ih / W_hh / b_ih / b_hh stack the reset, update and candidate blocks in that order.
    """
    D, n, A, H = cfg["D"], cfg["n"], cfg["A"], cfg["H"]
    I = D + n + A
    rng = np.random.Generator(np.random.Philox(key=(cfg["seed"] if seed is None else seed) + (4 << 40)))

    def xavier(fan_out, fan_in):
        a = math.sqrt(6.0 / (fan_in + fan_out))
        return rng.uniform(-a, a, size=(fan_out, fan_in)).astype(np.float32)

    def bias(m, fan_in):
        b = bias_scale / math.sqrt(fan_in)
        return rng.uniform(-b, b, size=(m,)).astype(np.float32)

    return dict(W1=xavier(H, I), b1=bias(H, I), W_ih=xavier(3 * H, H), b_ih=bias(3 * H, H),
                W_hh=xavier(3 * H, H), b_hh=bias(3 * H, H), W2=xavier(A, H), b2=bias(A, H))


def typed(cfg: dict, agent_type=None) -> dict:
    """The same workload with one network per unit type: ``agent_type`` lists every agent's type (default: the two
    types of the workload's typed feature blocks - agents [0, n_type0) type 0, the others type 1)."""
    c = dict(cfg)
    if agent_type is None:
        n0 = cfg["env"]["n_type0"]
        assert 0 < n0 < cfg["n"], "the workload has no unit types of its own: pass agent_type"
        agent_type = [0] * n0 + [1] * (cfg["n"] - n0)
    assert len(agent_type) == cfg["n"] and sorted(set(agent_type)) == list(range(max(agent_type) + 1))
    c["agent_type"] = [int(t) for t in agent_type]
    c["name"] = cfg.get("name", "cfg") + "_typed"
    return c


def make_weights_typed(cfg: dict, seed: int | None = None) -> list:
    """One network per unit type of ``typed(cfg)``, each drawn like ``make_weights`` from a seed of its own."""
    base = cfg["seed"] if seed is None else seed
    return [make_weights(cfg, seed=base + 7919 * (k + 1)) for k in range(max(cfg["agent_type"]) + 1)]

"""Pins of the oracle's per-type agent networks (heterogeneous teams: Table I lists a scenario whose team mixes two
unit types).  The arithmetic of one row is the single-network forward pinned in test_oracle_pins.py; what is pinned
here is which network decides for which agent."""
import math

import numpy as np
import torch

import oracle
from paper_2205_05248_b200 import workloads
from test_oracle_pins import _torch_reference


def _roll(cfg, w, T=None, **kw):
    sess = oracle.Session(cfg, w, np.arange(cfg["E"]), **kw)
    tr = sess.rollout(cfg["env"], cfg["T"] if T is None else T, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    return sess, tr


def test_identical_networks_per_type_equal_the_shared_network_bit_for_bit():
    base = workloads.config(3, E=6)
    base["T"] = 40
    w = workloads.make_weights(base)
    shared, tr_s = _roll(base, w)
    cfg = workloads.typed(base)
    assert cfg["agent_type"] == [0, 0, 1, 1, 1]
    typed, tr_t = _roll(cfg, [w, w])
    for k in tr_s:
        assert np.array_equal(tr_s[k], tr_t[k]), k
    for k in shared.ring:
        assert np.array_equal(shared.ring[k], typed.ring[k]), k
    assert np.array_equal(shared.h, typed.h) and np.array_equal(shared.counters, typed.counters)


def test_each_agent_is_decided_by_the_network_of_its_type():
    """Every traced Q row of a typed rollout equals the single-network forward with the agent's own type's weights
    on the recorded observation, the last action taken and the carried hidden state - and not the other type's."""
    cfg = workloads.typed(workloads.small_config(E=3, n=5, D=7, A=4, H=8, C=6, L=5, T=9, env=dict(n_type0=2)),
                          agent_type=[1, 0, 2, 0, 1])
    ws = workloads.make_weights_typed(cfg)
    assert len(ws) == 3
    sess, tr = _roll(cfg, ws)
    E, n, H = cfg["E"], cfg["n"], cfg["H"]
    h = np.zeros((E, n, H), np.float32)
    last = -np.ones((E, n), np.int64)
    wrong = 0
    for t in range(cfg["T"]):
        for e in range(E):
            for i in range(n):
                k = cfg["agent_type"][i]
                q, h1 = oracle.agent_forward(cfg, ws[k], tr["obs"][t, e, i], i, int(last[e, i]), h[e, i])
                assert np.array_equal(q, tr["q"][t, e, i]) and np.array_equal(h1, tr["h"][t, e, i])
                q_other, _ = oracle.agent_forward(cfg, ws[(k + 1) % 3], tr["obs"][t, e, i], i, int(last[e, i]), h[e, i])
                wrong += int(not np.array_equal(q_other, q))
                h[e, i] = h1
                last[e, i] = tr["action"][t, e, i]
            if tr["done"][t, e] or tr["pos"][t, e] + 1 == cfg["L"]:
                h[e] = 0
                last[e] = -1
    assert wrong == cfg["T"] * E * n          # the choice of network matters in every row


def test_two_scalar_networks_by_hand():
    """D = A = H = 1, two agents of two types, each worked out by hand from its own six numbers."""
    cfg = workloads.typed(workloads.small_config(D=1, n=2, A=1, H=1, E=1, C=1, L=4, T=1, eps_start=0.0, eps_end=0.0),
                          agent_type=[0, 1])
    f = lambda v: float(np.float32(v))
    nets = []
    for (wo, wid0, wid1, wla, b1, wi, bi, wh, bh, w2, b2) in (
            (0.5, -0.25, 0.1, 0.75, 0.1, (0.3, -0.6, 0.9), (0.01, 0.02, 0.03), (-0.2, 0.4, 0.7), (0.04, 0.05, 0.06), 2.0, -1.0),
            (-0.4, 0.2, 0.35, -0.5, 0.3, (0.8, 0.1, -0.7), (0.07, -0.02, 0.05), (0.6, -0.3, 0.2), (-0.01, 0.03, 0.02), -1.5, 0.25)):
        nets.append(dict(W1=np.array([[wo, wid0, wid1, wla]], np.float32), b1=np.array([b1], np.float32),
                         W_ih=np.array([[v] for v in wi], np.float32), b_ih=np.array(bi, np.float32),
                         W_hh=np.array([[v] for v in wh], np.float32), b_hh=np.array(bh, np.float32),
                         W2=np.array([[w2]], np.float32), b2=np.array([b2], np.float32)))
    obs = np.array([[[0.8], [-0.6]]], np.float32)
    sess = oracle.Session(cfg, nets, np.arange(1))
    sess.h[:] = np.array([[[-0.3], [0.45]]], np.float32)
    _, tr = sess.step(obs, np.ones((1, 2, 1), np.uint8), np.zeros(1, np.float32), np.zeros(1, np.uint8), 0.0,
                      trace=("q", "h"))
    for i, (o, h) in enumerate(((0.8, -0.3), (-0.6, 0.45))):
        w = nets[i]
        W1, wi, bi, wh, bh = w["W1"][0], w["W_ih"][:, 0], w["b_ih"], w["W_hh"][:, 0], w["b_hh"]
        y = f(max(0.0, f(w["b1"][0]) + f(W1[0]) * f(o) + f(W1[1 + i])))            # no last action at episode start
        r = 1 / (1 + math.exp(-(f(bi[0]) + f(wi[0]) * y + f(bh[0]) + f(wh[0]) * f(h))))
        z = 1 / (1 + math.exp(-(f(bi[1]) + f(wi[1]) * y + f(bh[1]) + f(wh[1]) * f(h))))
        c = math.tanh(f(bi[2]) + f(wi[2]) * y + r * (f(bh[2]) + f(wh[2]) * f(h)))
        hn = f((1 - z) * c + z * f(h))
        qq = f(f(w["b2"][0]) + f(w["W2"][0, 0]) * hn)
        assert abs(tr["h"][0, i, 0] - hn) <= 1e-7 and abs(tr["q"][0, i, 0] - qq) <= 2e-7


def test_typed_step_matches_float64_library_cells_per_type():
    """Workload 3's team (two units of one type, three of the other): one float64 torch Linear/GRUCell stack per
    type; every agent's row of a typed step equals the stack of its type."""
    cfg = workloads.typed(dict(workloads.config(3, E=2), precision="fp32"))
    ws = workloads.make_weights_typed(cfg)
    rng = np.random.default_rng(3)
    E, n, D, A, H = cfg["E"], cfg["n"], cfg["D"], cfg["A"], cfg["H"]
    obs = rng.uniform(-1, 1, (E, n, D)).astype(np.float32)
    h0 = rng.uniform(-1, 1, (E, n, H)).astype(np.float32)
    last = rng.integers(-1, A, (E, n)).astype(np.int32)
    sess = oracle.Session(cfg, ws, np.arange(E))
    sess.h[:] = h0
    sess.last_action[:] = last
    _, tr = sess.step(obs, np.ones((E, n, A), np.uint8), np.zeros(E, np.float32), np.zeros(E, np.uint8), 0.0,
                      trace=("q", "h"))
    for e in range(E):
        for i in range(n):
            qr, hr = _torch_reference(cfg, ws[cfg["agent_type"][i]], obs[e, i], i, int(last[e, i]), h0[e, i])
            assert np.max(np.abs(tr["h"][e, i] - hr)) <= 1.5e-7
            assert np.max(np.abs(tr["q"][e, i] - qr)) <= 1e-6 * max(1.0, np.max(np.abs(qr)))

"""Pins of the CPU oracle against facts that do not come from the oracle itself.

Each test names the mistake it is meant to catch.  Nothing here needs a GPU.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2205_05248_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------------------------------
# Philox4x32-10
# --------------------------------------------------------------------------------------------------
def _kat_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        rows.append([[int(x, 16) for x in part.split()] for part in line.split("|")])
    return rows


def test_philox_known_answers():
    """Published known-answer vectors of the generator's authors (wrong constant, wrong word order,
    key bumped at the wrong time, nine instead of ten rounds all fail here)."""
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert list(oracle.philox4x32_10(ctr, key)) == out


def _philox_bigint(ctr, key, rounds=10):
    """Second implementation with Python integers, written from the published round function."""
    c = list(ctr)
    k = list(key)
    for r in range(rounds):
        if r:
            k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
    return c


def test_philox_matches_bigint_reimplementation():
    rows = _kat_rows()
    for ctr, key, out in rows:   # the re-implementation itself is pinned by the same vectors
        assert _philox_bigint(ctr, key) == out
    rng = np.random.default_rng(1)
    for _ in range(2000):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4)]
        key = [int(x) for x in rng.integers(0, 2**32, 2)]
        assert list(oracle.philox4x32_10(ctr, key)) == _philox_bigint(ctr, key)


def test_uniform24_is_top_24_bits():
    assert oracle.uniform24(0) == 0.0
    assert oracle.uniform24(0xFF) == 0.0                       # low 8 bits are dropped
    assert oracle.uniform24(0x100) == 2.0 ** -24
    assert oracle.uniform24(0xFFFFFFFF) == 1.0 - 2.0 ** -24    # never reaches 1
    assert oracle.uniform24(0x80000000) == 0.5


# --------------------------------------------------------------------------------------------------
# bfloat16 rounding
# --------------------------------------------------------------------------------------------------
def test_bf16_round_all_bf16_values_are_fixed_points():
    bits = (np.arange(1 << 16, dtype=np.uint32) << 16)
    vals = bits.view(np.float32)
    for v in vals[::17]:
        if math.isnan(v):
            continue
        r = oracle.bf16_round(float(v))
        assert np.float32(r).view(np.uint32) == np.float32(v).view(np.uint32)


def test_bf16_round_ties_to_even_and_library_agreement():
    def f(bits):
        return float(np.uint32(bits).view(np.float32))
    # exactly half-way between two bf16 numbers: goes to the one with an even last bit
    assert oracle.bf16_round(f(0x3F808000)) == f(0x3F800000)   # 1 + 2^-8  -> 1 (even)
    assert oracle.bf16_round(f(0x3F818000)) == f(0x3F820000)   # odd below -> rounds up to even
    assert oracle.bf16_round(f(0x3F808001)) == f(0x3F810000)   # just above half -> up
    assert oracle.bf16_round(f(0x3F807FFF)) == f(0x3F800000)   # just below half -> down
    assert oracle.bf16_round(-f(0x3F808001)) == -f(0x3F810000)
    assert oracle.bf16_round(f(0x7F7FFFFF)) == float("inf")    # overflow rounds to infinity
    # library special case: torch's float32 -> bfloat16 conversion is round-to-nearest-even
    x = torch.randn(5000, dtype=torch.float32, generator=torch.Generator().manual_seed(3)) * 7
    want = x.to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.bf16_round(float(v)) for v in x.numpy()], np.float32)
    assert np.array_equal(got, want)


# --------------------------------------------------------------------------------------------------
# Agent network
# --------------------------------------------------------------------------------------------------
def _zero_weights(cfg):
    D, n, A, H = cfg["D"], cfg["n"], cfg["A"], cfg["H"]
    I = D + n + A
    z = lambda *s: np.zeros(s, np.float32)
    return dict(W1=z(H, I), b1=z(H), W_ih=z(3 * H, H), b_ih=z(3 * H), W_hh=z(3 * H, H), b_hh=z(3 * H),
                W2=z(A, H), b2=z(A))


def test_gru_zero_matrices_closed_form():
    """All matrices zero: r = sigma(b_ir+b_hr), z = sigma(b_iz+b_hz), c = tanh(b_in + r b_hn),
    h' = (1-z) c + z h, Q = b2.  Catches a missing bias, the reset gate applied to the wrong term,
    and the blend written the other way round."""
    cfg = workloads.small_config(H=4, A=3)
    w = _zero_weights(cfg)
    H = 4
    w["b_ih"][:] = np.array([0.3] * H + [-0.7] * H + [0.2] * H, np.float32)
    w["b_hh"][:] = np.array([0.1] * H + [0.4] * H + [-0.9] * H, np.float32)
    w["b2"][:] = [1.0, -2.0, 0.5]
    h0 = np.array([0.5, -0.25, 0.0, 1.0], np.float32)
    q, h1 = oracle.agent_forward(cfg, w, np.ones(cfg["D"], np.float32), 1, 2, h0)
    sig = lambda v: 1.0 / (1.0 + math.exp(-v))
    r = sig(np.float32(0.3) + np.float32(0.1))
    z = sig(float(np.float32(-0.7)) + float(np.float32(0.4)))
    c = math.tanh(float(np.float32(0.2)) + r * float(np.float32(-0.9)))
    want = (1 - z) * c + z * h0.astype(np.float64)
    assert np.allclose(h1, want, rtol=0, atol=1e-7)
    assert np.array_equal(q, w["b2"])
    # with b = 0 everywhere: r = z = 1/2, c = 0, h' = h/2
    w2 = _zero_weights(cfg)
    _, h2 = oracle.agent_forward(cfg, w2, np.ones(cfg["D"], np.float32), 0, -1, h0)
    assert np.array_equal(h2, h0 / 2)


def test_gru_saturated_update_gate():
    """z -> 1 keeps the old state, z -> 0 replaces it by the candidate."""
    cfg = workloads.small_config(H=4, A=3)
    w = workloads.make_weights(cfg)
    h0 = np.array([0.5, -0.25, 0.125, 0.9], np.float32)
    obs = np.linspace(-1, 1, cfg["D"]).astype(np.float32)
    H = 4
    w_keep = {k: v.copy() for k, v in w.items()}
    w_keep["b_ih"][H:2 * H] = 60.0
    _, h1 = oracle.agent_forward(cfg, w_keep, obs, 0, -1, h0)
    assert np.array_equal(h1, h0)
    w_new = {k: v.copy() for k, v in w.items()}
    w_new["b_ih"][H:2 * H] = -60.0
    _, h2 = oracle.agent_forward(cfg, w_new, obs, 0, -1, h0)
    assert np.all(np.abs(h2) <= 1.0) and not np.allclose(h2, h0)
    # the candidate does not depend on the update-gate rows at all
    w_new2 = {k: v.copy() for k, v in w_new.items()}
    w_new2["W_ih"][H:2 * H] *= -3.0
    _, h3 = oracle.agent_forward(cfg, w_new2, obs, 0, -1, h0)
    assert np.allclose(h2, h3, atol=1e-7)


def test_scalar_network_by_hand():
    """D = n = A = H = 1, worked out step by step.
    x = [o, 1, (last==0)];  y = relu(w_o o + w_id + w_la + b1);  the GRU and fc2 are scalars."""
    cfg = workloads.small_config(D=1, n=1, A=1, H=1, E=1, C=1)
    w = dict(W1=np.array([[0.5, -0.25, 0.75]], np.float32), b1=np.array([0.1], np.float32),
             W_ih=np.array([[0.3], [-0.6], [0.9]], np.float32), b_ih=np.array([0.01, 0.02, 0.03], np.float32),
             W_hh=np.array([[-0.2], [0.4], [0.7]], np.float32), b_hh=np.array([0.04, 0.05, 0.06], np.float32),
             W2=np.array([[2.0]], np.float32), b2=np.array([-1.0], np.float32))
    o, h = 0.8, -0.3
    f = lambda v: float(np.float32(v))
    for last in (-1, 0):
        y = max(0.0, f(0.1) + f(0.5) * f(o) + f(-0.25) + (f(0.75) if last == 0 else 0.0))
        y = f(y)
        r = 1 / (1 + math.exp(-(f(0.01) + f(0.3) * y + f(0.04) + f(-0.2) * f(h))))
        z = 1 / (1 + math.exp(-(f(0.02) + f(-0.6) * y + f(0.05) + f(0.4) * f(h))))
        c = math.tanh(f(0.03) + f(0.9) * y + r * (f(0.06) + f(0.7) * f(h)))
        hn = f((1 - z) * c + z * f(h))
        qq = f(-1.0 + 2.0 * hn)
        q, h1 = oracle.agent_forward(cfg, w, np.array([o], np.float32), 0, last, np.array([h], np.float32))
        assert abs(h1[0] - hn) <= 1e-7 and abs(q[0] - qq) <= 2e-7


def _torch_reference(cfg, w, obs, agent, last, h0, lowp=False):
    """float64 torch.nn.Linear / GRUCell with the same weights (library special case)."""
    D, n, A, H = cfg["D"], cfg["n"], cfg["A"], cfg["H"]
    I = D + n + A
    rb = (lambda t: t.to(torch.bfloat16).to(torch.float64)) if lowp else (lambda t: t.to(torch.float64))
    fc1 = torch.nn.Linear(I, H).double()
    gru = torch.nn.GRUCell(H, H).double()
    fc2 = torch.nn.Linear(H, A).double()
    T = lambda k: torch.from_numpy(w[k])
    with torch.no_grad():
        fc1.weight.copy_(rb(T("W1"))); fc1.bias.copy_(T("b1").double())
        gru.weight_ih.copy_(rb(T("W_ih"))); gru.bias_ih.copy_(T("b_ih").double())
        gru.weight_hh.copy_(rb(T("W_hh"))); gru.bias_hh.copy_(T("b_hh").double())
        fc2.weight.copy_(rb(T("W2"))); fc2.bias.copy_(T("b2").double())
        x = torch.zeros(I, dtype=torch.float64)
        x[:D] = rb(torch.from_numpy(obs))
        x[D + agent] = 1.0
        if last >= 0:
            x[D + n + last] = 1.0
        y = torch.relu(fc1(x))
        h0t = torch.from_numpy(h0)
        if not lowp:
            h1 = gru(y[None], h0t.double()[None])[0]
            q = fc2(h1.float().double())
        else:
            # operands rounded to bf16; the blend uses the unrounded previous state
            yq = rb(y.float())
            hq = rb(h0t)
            gi = gru.weight_ih @ yq + gru.bias_ih
            gh = gru.weight_hh @ hq + gru.bias_hh
            r = torch.sigmoid(gi[:H] + gh[:H])
            z = torch.sigmoid(gi[H:2 * H] + gh[H:2 * H])
            c = torch.tanh(gi[2 * H:] + r * gh[2 * H:])
            h1 = (1 - z) * c + z * h0t.double()
            q = fc2(rb(h1.float()))
    return q.numpy(), h1.numpy()


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_network_matches_float64_library_cells(k):
    """torch.nn.Linear + torch.nn.GRUCell in float64 on the experiment shapes.  Catches a transposed
    weight, swapped gate blocks, a wrong one-hot column offset, a dropped term."""
    cfg = workloads.config(k)
    cfg = dict(cfg, precision="fp32")
    w = workloads.make_weights(cfg)
    rng = np.random.default_rng(k)
    for trial in range(6):
        obs = rng.uniform(-1, 1, cfg["D"]).astype(np.float32)
        h0 = rng.uniform(-1, 1, cfg["H"]).astype(np.float32)
        agent = int(rng.integers(cfg["n"]))
        last = int(rng.integers(-1, cfg["A"]))
        q, h1 = oracle.agent_forward(cfg, w, obs, agent, last, h0)
        qr, hr = _torch_reference(cfg, w, obs, agent, last, h0)
        assert np.max(np.abs(h1 - hr)) <= 1.5e-7     # one float rounding of a value in [-1, 1]
        assert np.max(np.abs(q - qr)) <= 1e-6 * max(1.0, np.max(np.abs(qr)))


def test_bf16_mode_rounds_exactly_the_stated_operands():
    cfg = dict(workloads.config(2), precision="bf16")
    w = workloads.make_weights(cfg)
    rng = np.random.default_rng(7)
    for trial in range(4):
        obs = rng.normal(0, 1, cfg["D"]).astype(np.float32)
        h0 = rng.uniform(-1, 1, cfg["H"]).astype(np.float32)
        q, h1 = oracle.agent_forward(cfg, w, obs, 3, 5, h0)
        qr, hr = _torch_reference(cfg, w, obs, 3, 5, h0, lowp=True)
        assert np.max(np.abs(h1 - hr)) <= 1.5e-7
        assert np.max(np.abs(q - qr)) <= 1e-6 * max(1.0, np.max(np.abs(qr)))
        q32, _ = oracle.agent_forward(dict(cfg, precision="fp32"), w, obs, 3, 5, h0)
        assert 1e-6 < np.max(np.abs(q - q32)) < 5e-2   # the rounding is really applied, and is small


# --------------------------------------------------------------------------------------------------
# Masked greedy choice, tie rule, epsilon draw
# --------------------------------------------------------------------------------------------------
def _brute_greedy(q, avail):
    cand = [a for a in range(len(q)) if avail[a]]
    if not cand:
        return 0
    m = max(np.float32(q[a]) for a in cand)
    thr = np.float32(m) - np.float32(1e-4)
    return min(a for a in cand if np.float32(q[a]) >= thr)


def test_greedy_brute_force_all_masks():
    rng = np.random.default_rng(11)
    A = 9
    for trial in range(4):
        q = rng.normal(0, 1, A).astype(np.float32)
        for mask in range(1 << A):
            avail = np.array([(mask >> a) & 1 for a in range(A)], np.uint8)
            a, ex, u, na = oracle.select_action(q, avail, 0.0, 5, trial, mask, 0)
            assert ex == 0
            if mask == 0:
                assert (a, na) == (0, 1)
            else:
                assert na == 0 and avail[a] == 1
                assert a == _brute_greedy(q, avail)


def test_greedy_tie_rule_constructed():
    """Gaps of 0, 0.5e-4 (inside the band: lowest index wins) and 1.5e-4 (outside: the maximum wins)."""
    A = 6
    for i in range(A):
        for j in range(i + 1, A):
            for gap, want in ((0.0, i), (0.5e-4, i), (1.5e-4, j)):
                q = np.full(A, -5.0, np.float32)
                q[j] = 1.0
                q[i] = np.float32(1.0) - np.float32(gap)
                a, *_ = oracle.select_action(q, np.ones(A, np.uint8), 0.0, 1, 0, 0, 0)
                assert a == want
                # the lower-index candidate masked out: the other one is chosen
                av = np.ones(A, np.uint8)
                av[i] = 0
                a, *_ = oracle.select_action(q, av, 0.0, 1, 0, 0, 0)
                assert a == j
    # an unavailable action never wins even with the largest Q
    q = np.array([0.0, 9.0, 1.0], np.float32)
    a, *_ = oracle.select_action(q, np.array([1, 0, 1], np.uint8), 0.0, 1, 0, 0, 0)
    assert a == 2


def test_epsilon_draw_keying_and_pick():
    """u is word 0 of block (t, e, i, tag 0) under key = seed; the pick is floor(w1 K / 2^32)."""
    seed = 0x123456789ABCDEF0
    A = 7
    avail = np.array([1, 0, 1, 1, 0, 1, 1], np.uint8)
    idx = [a for a in range(A) if avail[a]]
    q = np.arange(A, dtype=np.float32)
    for (t, e, i) in [(0, 0, 0), (5, 17, 2), (1000, 65535, 7), (2**31, 3, 1)]:
        w = _philox_bigint([t, e, i, 0], [seed & 0xFFFFFFFF, seed >> 32])
        u = (w[0] >> 8) * 2.0 ** -24
        a, ex, uo, _ = oracle.select_action(q, avail, 1.0, seed, t, e, i)
        assert uo == u and ex == 1
        assert a == idx[(w[1] * len(idx)) >> 32]
        a0, ex0, _, _ = oracle.select_action(q, avail, 0.0, seed, t, e, i)
        assert ex0 == 0 and a0 == 6
        # explore iff u < eps, strictly
        eps_just_above = float(np.nextafter(np.float32(u), np.float32(2)))
        assert oracle.select_action(q, avail, eps_just_above, seed, t, e, i)[1] == 1
        assert oracle.select_action(q, avail, float(np.float32(u)), seed, t, e, i)[1] == 0


def test_epsilon_statistics():
    """Explore count ~ Binomial(N, eps); random picks uniform over the available actions."""
    A = 8
    avail = np.array([1, 1, 0, 1, 1, 1, 0, 1], np.uint8)
    q = np.zeros(A, np.float32)
    N, eps = 20000, 0.3
    n_ex = 0
    hist = np.zeros(A)
    for t in range(N):
        a, ex, _, _ = oracle.select_action(q, avail, eps, 99, t, t % 13, t % 5)
        assert avail[a]
        n_ex += ex
        if ex:
            hist[a] += 1
    assert abs(n_ex - N * eps) < 4 * math.sqrt(N * eps * (1 - eps))
    K = int(avail.sum())
    exp = n_ex / K
    chi2 = sum((hist[a] - exp) ** 2 / exp for a in range(A) if avail[a])
    assert hist[avail == 0].sum() == 0
    assert chi2 < 25.0          # 5 degrees of freedom, far tail


def test_eps_schedule():
    assert oracle.eps_at(0.05, 0.05, 0, 7) == float(np.float32(0.05))
    assert oracle.eps_at(1.0, 0.05, 255, 0) == 1.0
    assert oracle.eps_at(1.0, 0.05, 255, 255) == float(np.float32(0.05))   # reaches the end value exactly
    assert oracle.eps_at(1.0, 0.05, 255, 999) == float(np.float32(0.05))   # and stays there
    mid = oracle.eps_at(1.0, 0.0, 10, 5)
    assert mid == 0.5
    vals = [oracle.eps_at(1.0, 0.05, 255, t) for t in range(256)]
    assert all(a > b for a, b in zip(vals, vals[1:]))


# --------------------------------------------------------------------------------------------------
# Synthetic environment streams
# --------------------------------------------------------------------------------------------------
def test_env_stream_definitions():
    """Each stream re-derived from the big-integer Philox: catches a wrong tag, block or word."""
    cfg = workloads.config(2)
    env = cfg["env"]
    key = [env["seed"] & 0xFFFFFFFF, env["seed"] >> 32]
    t, e = 37, 513
    obs, avail, reward, done = oracle.env_emit(cfg, env, t, e)
    w = _philox_bigint([t, e, 0, 1], key)
    assert done == int((w[0] >> 8) < env["done_thresh24"])

    def ih12(b1, b2):
        hw = []
        for x in b1 + b2[:2]:
            hw += [x & 0xFFFF, x >> 16]
        return (sum(hw) - 393210) / 65536.0
    assert reward == ih12(_philox_bigint([t, e, 1 << 16, 1], key), _philox_bigint([t, e, 2 << 16, 1], key))
    for i in (0, 7):
        for a in (0, 1, 5, 13):
            if a == 0:
                assert avail[i, a] == 1
            else:
                ww = _philox_bigint([t, e, i | ((a // 4) << 16), 2], key)
                assert avail[i, a] == int((ww[a % 4] >> 8) < env["avail_thresh_first"])
        for k in (0, 3, 79):
            v = ih12(_philox_bigint([t, e, i | ((2 * k) << 16), 3], key),
                     _philox_bigint([t, e, i | ((2 * k + 1) << 16), 3], key))
            assert obs[i, k] == np.float32(min(3.0, max(-3.0, v)))
    # uniform law
    cfg1 = workloads.config(1)
    obs, avail, _, _ = oracle.env_emit(cfg1, cfg1["env"], 3, 5)
    key1 = [cfg1["env"]["seed"] & 0xFFFFFFFF, cfg1["env"]["seed"] >> 32]
    for i, k in ((0, 0), (2, 29), (1, 6)):
        ww = _philox_bigint([3, 5, i | ((k // 4) << 16), 3], key1)
        assert obs[i, k] == np.float32(((ww[k % 4] >> 8) - 2**23) / 2.0**23)


def test_env_stream_moments():
    cfg = workloads.config(2, E=64)
    env = cfg["env"]
    obs_all, av_all, rew, dn = [], [], [], []
    for t in range(40):
        for e in range(16):
            o, a, r, d = oracle.env_emit(cfg, env, t, e)
            obs_all.append(o); av_all.append(a); rew.append(r); dn.append(d)
    obs_all = np.stack(obs_all); av_all = np.stack(av_all); rew = np.array(rew)
    N = obs_all.size
    assert abs(obs_all.mean()) < 4 / math.sqrt(N)
    assert abs(obs_all.var() - 0.997) < 0.01          # unit variance, minus what the clip at 3 removes
    assert obs_all.max() <= 3.0 and obs_all.min() >= -3.0
    assert abs(rew.mean()) < 4 / math.sqrt(len(rew)) and abs(rew.var() - 1) < 0.25
    p = av_all[:, :, 1:].mean()
    M = av_all[:, :, 1:].size
    assert abs(p - 0.7) < 4 * math.sqrt(0.21 / M)
    assert av_all[:, :, 0].all()
    # uniform law and the two-probability mask of workload 4
    cfg4 = workloads.config(4)
    o4 = []; a4 = []
    for t in range(30):
        o, a, _, _ = oracle.env_emit(cfg4, cfg4["env"], t, 1234)
        o4.append(o); a4.append(a)
    o4 = np.stack(o4); a4 = np.stack(a4)
    assert abs(o4.mean()) < 4 * math.sqrt(1 / 3 / o4.size) and abs(o4.var() - 1 / 3) < 0.02
    assert -1.0 <= o4.min() and o4.max() < 1.0
    assert abs(a4[:, :, 1:6].mean() - 0.9) < 0.06 and abs(a4[:, :, 6:].mean() - 0.5) < 0.08
    # done rate
    cfgd = workloads.small_config()
    dn = [oracle.env_emit(cfgd, cfgd["env"], t, e)[3] for t in range(400) for e in range(4)]
    assert abs(np.mean(dn) - 0.15) < 4 * math.sqrt(0.15 * 0.85 / len(dn))


def test_env_typed_feature_blocks():
    cfg = workloads.config(3)
    obs, *_ = oracle.env_emit(cfg, cfg["env"], 9, 100)
    assert np.all(obs[:2, 64:80] == 0) and np.all(obs[2:, 48:64] == 0)      # the other type's block
    assert np.all(obs[:2, 48:64] != 0) and np.all(obs[2:, 64:80] != 0)
    assert np.all(obs[:, :48] != 0)

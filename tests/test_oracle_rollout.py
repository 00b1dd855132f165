"""Invariants of the oracle's rollout: what the paper's prose fixes about the loop, checked on the oracle.

* hidden state is private to one (environment, agent) pair (Sec. III-A, Fig. 3);
* an episode end resets the environment's recurrent state (Algorithm 1: reset at episode start);
* every step is recorded and whole episodes are handed over (Algorithm 1).
"""
import numpy as np

import oracle
from paper_2205_05248_b200 import workloads


def _session(cfg, env_ids=None, **kw):
    w = workloads.make_weights(cfg)
    ids = np.arange(cfg["E"]) if env_ids is None else np.asarray(env_ids)
    return oracle.Session(cfg, w, ids, **kw), w


def _roll(sess, cfg, T=None, **kw):
    return sess.rollout(cfg["env"], cfg["T"] if T is None else T, cfg["eps_start"], cfg["eps_end"],
                        cfg["anneal_steps"], **kw)


def test_hidden_state_isolation_subset_and_permutation():
    """An environment's trajectory does not depend on which other environments are stepped with it."""
    cfg = workloads.small_config(E=6, C=12, T=12)
    full, _ = _session(cfg)
    tr = _roll(full, cfg)
    ids = [4, 1, 5]
    part, _ = _session(cfg, ids)
    trp = _roll(part, cfg)
    for k in ("obs", "avail", "q", "h", "action", "explore", "u", "slot", "pos", "reward", "done"):
        assert np.array_equal(tr[k][:, ids], trp[k]), k
    assert np.array_equal(full.h[ids], part.h)
    S = full.S
    for x, e in enumerate(ids):
        for k in ("obs", "q", "action", "slot_epid", "slot_len", "slot_complete"):
            assert np.array_equal(full.ring[k][e * S:(e + 1) * S], part.ring[k][x * S:(x + 1) * S]), k


def test_threads_do_not_change_the_result():
    cfg = workloads.small_config(E=7, C=14, T=10)
    a, _ = _session(cfg, n_threads=1)
    b, _ = _session(cfg, n_threads=3)
    ta, tb = _roll(a, cfg), _roll(b, cfg)
    for k in ta:
        assert np.array_equal(ta[k], tb[k]), k
    assert np.array_equal(a.counters, b.counters)
    for k in a.ring:
        assert np.array_equal(a.ring[k], b.ring[k]), k


def test_done_every_step_makes_every_step_a_first_step():
    cfg = workloads.small_config(E=3, C=3 * 16, L=4, T=10, env=dict(done_thresh24=1 << 24))
    s, w = _session(cfg)
    tr = _roll(s, cfg)
    assert tr["done"].all() and (tr["pos"] == 0).all()
    for t in range(cfg["T"]):
        for e in range(cfg["E"]):
            for i in range(cfg["n"]):
                q, h = oracle.agent_forward(cfg, w, tr["obs"][t, e, i], i, -1, np.zeros(cfg["H"], np.float32))
                assert np.array_equal(q, tr["q"][t, e, i]) and np.array_equal(h, tr["h"][t, e, i])
    assert np.all(s.h == 0) and np.all(s.last_action == -1)
    assert np.array_equal(s.ep_count, np.full(3, 10))


def test_no_done_no_reset_and_truncation_at_ring_length():
    cfg = workloads.small_config(E=2, C=4, L=5, T=12, env=dict(done_thresh24=0))
    s, w = _session(cfg)
    tr = _roll(s, cfg)
    assert not tr["done"].any()
    assert np.array_equal(tr["pos"][:, 0], np.arange(12) % 5)          # truncated every L steps
    assert s.counters[oracle.CNT_TRUNCATED] == 2 * 2 and s.counters[oracle.CNT_EPISODES] == 4
    # the recurrent input of step t is the stored output of step t-1, except right after a truncation
    for t in range(1, 12):
        prev_h = tr["h"][t - 1, 0, 1] if t % 5 else np.zeros(cfg["H"], np.float32)
        last = tr["action"][t - 1, 0, 1] if t % 5 else -1
        q, h = oracle.agent_forward(cfg, w, tr["obs"][t, 0, 1], 1, int(last), prev_h)
        assert np.array_equal(q, tr["q"][t, 0, 1])
    # a truncated episode is complete but its last done flag is 0
    S = s.S
    closed = np.nonzero(s.ring["slot_complete"])[0]
    assert len(closed) > 0
    for rs in closed:
        assert s.ring["slot_len"][rs] == 5 and s.ring["done"][rs, 4] == 0


def test_ring_bookkeeping_invariants():
    cfg = workloads.small_config(E=5, C=20, L=6, T=40)
    s, _ = _session(cfg)
    tr = _roll(s, cfg)
    E, S, L, T = cfg["E"], s.S, cfg["L"], cfg["T"]
    closes = 0
    for e in range(E):
        pos, k = 0, 0
        for t in range(T):
            assert tr["pos"][t, e] == pos
            assert tr["slot"][t, e] == e * S + (k % S)
            if tr["done"][t, e] or pos + 1 == L:
                pos, k = 0, k + 1
                closes += 1
            else:
                pos += 1
        assert s.ep_count[e] == k and s.pos[e] == pos and s.slot[e] == e * S + (k % S)
        # headers of this env's sub-ring: ids are k*E+e for the most recent episodes
        for ls in range(S):
            rs = e * S + ls
            epid = s.ring["slot_epid"][rs]
            if epid >= 0:
                assert epid % E == e and (epid // E) % S == ls
                kk = epid // E
                assert (kk < k and s.ring["slot_complete"][rs] == 1) or (kk == k and s.ring["slot_complete"][rs] == 0)
    assert s.counters[oracle.CNT_EPISODES] == closes
    assert s.counters[oracle.CNT_STEPS] == E * cfg["n"] * T
    # rows still in the ring equal the traced rows that wrote them (last writer wins)
    last_writer = {}
    for t in range(T):
        for e in range(E):
            last_writer[(tr["slot"][t, e], tr["pos"][t, e])] = (t, e)
    for (slot, pos), (t, e) in last_writer.items():
        assert np.array_equal(s.ring["obs"][slot, pos], tr["obs"][t, e])
        assert np.array_equal(s.ring["q"][slot, pos], tr["q"][t, e])
        assert np.array_equal(s.ring["action"][slot, pos], tr["action"][t, e])
        assert np.array_equal(s.ring["avail"][slot, pos], tr["avail"][t, e])
        assert s.ring["reward"][slot, pos] == tr["reward"][t, e] and s.ring["done"][slot, pos] == tr["done"][t, e]


def test_chosen_action_is_always_available_and_explore_rate():
    cfg = workloads.small_config(E=16, C=16, L=64, T=50, eps_start=0.25, eps_end=0.25)
    s, _ = _session(cfg)
    tr = _roll(s, cfg)
    a = tr["action"]
    assert np.take_along_axis(tr["avail"], a[..., None], axis=-1).all()
    N = a.size
    assert abs(tr["explore"].mean() - 0.25) < 4 * np.sqrt(0.25 * 0.75 / N)
    assert np.array_equal(tr["action"], tr["action_free"])
    assert s.counters[oracle.CNT_EXPLORE] == tr["explore"].sum()


def test_resume_two_halves_equal_one_rollout_and_step_api_equals_rollout():
    cfg = workloads.small_config(E=4, C=8, L=6, T=14, eps_start=1.0, eps_end=0.1, anneal_steps=13)
    one, _ = _session(cfg)
    tr = _roll(one, cfg)
    two, _ = _session(cfg)
    t1 = _roll(two, cfg, T=6)
    t2 = _roll(two, cfg, T=8)
    for k in tr:
        assert np.array_equal(tr[k], np.concatenate([t1[k], t2[k]])), k
    for k in one.ring:
        assert np.array_equal(one.ring[k], two.ring[k]), k
    # the step call fed with the synthetic environment's outputs reproduces the rollout
    st, _ = _session(cfg)
    for t in range(cfg["T"]):
        eps = oracle.eps_at(cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"], t)
        acts, _ = st.step(tr["obs"][t], tr["avail"][t], tr["reward"][t], tr["done"][t], eps)
        assert np.array_equal(acts, tr["action"][t])
    for k in one.ring:
        assert np.array_equal(one.ring[k], st.ring[k]), k
    assert np.array_equal(one.h, st.h)


def test_adopted_actions_feed_back_and_are_recorded():
    """The referee hook: an adopted action replaces the free choice in the record and in the next input."""
    cfg = workloads.small_config(E=2, C=2, L=32, T=6, env=dict(done_thresh24=0, avail_thresh_first=1 << 24,
                                                               avail_thresh_rest=1 << 24))
    free, w = _session(cfg)
    tr = _roll(free, cfg)
    adopt = tr["action"].copy()
    adopt[2, 1, 0] = (adopt[2, 1, 0] + 1) % cfg["A"]
    forced, _ = _session(cfg)
    tf = _roll(forced, cfg, adopt=adopt)
    assert np.array_equal(tf["action"], adopt)
    assert tf["action_free"][2, 1, 0] == tr["action"][2, 1, 0]
    assert np.array_equal(tf["q"][:3], tr["q"][:3])
    q, _ = oracle.agent_forward(cfg, w, tf["obs"][3, 1, 0], 0, int(adopt[2, 1, 0]), tf["h"][2, 1, 0])
    assert np.array_equal(q, tf["q"][3, 1, 0])
    assert not np.array_equal(tf["q"][3, 1, 0], tr["q"][3, 1, 0])
    assert np.array_equal(tf["q"][3, 0], tr["q"][3, 0])        # the other environment is untouched
    assert forced.ring["action"][forced.slot[1], 2, 0] == adopt[2, 1, 0]


def test_weight_switch_uses_the_new_network_from_the_next_step():
    """Sec. III-B: workers act with whatever model the learner last placed in the shared pool.  After a switch the
    Q rows are those of the new network applied (by the single-agent forward) to the carried-over hidden state."""
    cfg = workloads.small_config(E=3, C=6, L=5, T=9, env=dict(done_thresh24=0))
    sess, w0 = _session(cfg)
    w1 = workloads.make_weights(cfg, seed=cfg["seed"] + 5)
    t1 = _roll(sess, cfg, T=4)
    h_before, la_before = sess.h.copy(), sess.last_action.copy()
    sess.set_weights(w1)
    t2 = _roll(sess, cfg, T=1)
    for x in range(cfg["E"]):
        for i in range(cfg["n"]):
            q_new, _ = oracle.agent_forward(cfg, w1, t2["obs"][0, x, i], i, int(la_before[x, i]), h_before[x, i])
            q_old, _ = oracle.agent_forward(cfg, w0, t2["obs"][0, x, i], i, int(la_before[x, i]), h_before[x, i])
            assert np.allclose(t2["q"][0, x, i], q_new, rtol=1e-6, atol=1e-7)
            assert not np.allclose(t2["q"][0, x, i], q_old, rtol=1e-3, atol=1e-4)
    # the steps before the switch are those of a session that never switched
    plain, _ = _session(cfg)
    t0 = _roll(plain, cfg, T=4)
    assert all(np.array_equal(t0[k], t1[k]) for k in t0)


def test_subset_steps_touch_only_the_listed_environments_and_compose_to_a_full_step():
    """Asynchronous actors (Sec. III-A): a step over a list of environments is the full step restricted to them.
    Environments are independent, so stepping two disjoint halves under one step index equals one full step, and
    an environment that is not listed keeps its state and its part of the pool."""
    cfg = workloads.small_config(E=6, C=12, L=4, T=10, env=dict(done_thresh24=1 << 22))
    full, _ = _session(cfg)
    part, _ = _session(cfg)
    idle, _ = _session(cfg)
    a_ids, b_ids = np.array([4, 0, 3]), np.array([1, 5, 2])
    for t in range(cfg["T"]):
        outs = [oracle.env_emit(cfg, cfg["env"], t, e) for e in range(cfg["E"])]
        obs, avail, rew, done = (np.stack([o[k] for o in outs]) for k in range(4))
        acts, _ = full.step(obs, avail, rew, done, 0.2)
        before = (idle.h.copy(), idle.pos.copy(), {k: v.copy() for k, v in idle.ring.items()})
        acts_a, _ = part.step_subset(a_ids, obs[a_ids], avail[a_ids], rew[a_ids], done[a_ids], 0.2)
        part.t -= 1                                      # the second half belongs to the same step index
        acts_b, _ = part.step_subset(b_ids, obs[b_ids], avail[b_ids], rew[b_ids], done[b_ids], 0.2)
        assert np.array_equal(acts[a_ids], acts_a) and np.array_equal(acts[b_ids], acts_b)
        idle.step_subset(a_ids, obs[a_ids], avail[a_ids], rew[a_ids], done[a_ids], 0.2)
        S = idle.S
        for e in b_ids:                                  # not listed: nothing moved
            assert np.array_equal(idle.h[e], before[0][e]) and idle.pos[e] == before[1][e] == 0
            for k, v in idle.ring.items():
                assert np.array_equal(v[e * S:(e + 1) * S], before[2][k][e * S:(e + 1) * S]), k
    for k in ("h", "last_action", "slot", "pos", "ep_count"):
        assert np.array_equal(getattr(full, k), getattr(part, k)), k
    for k in full.ring:
        assert np.array_equal(full.ring[k], part.ring[k]), k
    assert np.array_equal(full.counters, part.counters)


def test_lagged_step_equals_the_synchronous_step_with_outcomes_one_call_late():
    """Algorithm 1: the reward and the end of the game are known after the action, so they reach the worker with the
    next observation.  Feeding each outcome one call late gives the same decisions, and every closed episode is
    recorded exactly as by the synchronous step (same records, same lengths, truncation at the slot length too)."""
    cfg = workloads.small_config(E=5, C=60, L=4, T=17, env=dict(done_thresh24=1 << 22))
    E, T = cfg["E"], cfg["T"]
    sync, _ = _session(cfg)
    lag, _ = _session(cfg)
    tr = _roll(sync, cfg)
    ids = np.arange(E)
    zr, zd = np.zeros(E, np.float32), np.zeros(E, np.uint8)
    for t in range(T):
        eps = oracle.eps_at(cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"], t)
        acts, ltr = lag.step_lagged(ids, tr["obs"][t], tr["avail"][t], tr["reward"][t - 1] if t else zr,
                                    tr["done"][t - 1] if t else zd, eps, trace=("q",))
        assert np.array_equal(acts, tr["action"][t]), t
        assert np.array_equal(ltr["q"], tr["q"][t]), t
    closed = lag.ring["slot_complete"] == 1
    assert closed.sum() >= 8 and (tr["done"].sum() > 0) and sync.counters[oracle.CNT_TRUNCATED] > 0
    for k in ("obs", "avail", "action", "q", "reward", "done", "slot_epid", "slot_len"):
        assert np.array_equal(lag.ring[k][closed], sync.ring[k][closed]), k
    # the synchronous session has also closed the episodes that end with the last step; the lagged one will on its
    # next call: until then the last outcome is missing and the cursor stands one past the record
    last_closes = (tr["done"][T - 1] != 0) | (tr["pos"][T - 1] + 1 == cfg["L"])
    assert np.array_equal(lag.ep_count + last_closes, sync.ep_count)
    assert np.array_equal(lag.pos[~last_closes], sync.pos[~last_closes])


def test_lagged_step_by_hand():
    """One environment, slot length 3: first call has nothing to commit; a 'done' closes the episode before the
    decision, which then starts from a zero hidden state and no last action in the next slot."""
    cfg = workloads.small_config(E=1, C=2, L=3, T=1)
    sess, w = _session(cfg)
    n, D, A, H = cfg["n"], cfg["D"], cfg["A"], cfg["H"]
    rng = np.random.default_rng(5)
    obs = rng.uniform(-1, 1, size=(5, 1, n, D)).astype(np.float32)
    avail = np.ones((1, n, A), np.uint8)
    one = lambda v, dt: np.array([v], dt)
    sess.step_lagged([0], obs[0], avail, one(9.0, np.float32), one(1, np.uint8), 0.0)       # outcome ignored
    assert sess.pos[0] == 1 and sess.ep_count[0] == 0 and sess.ring["slot_len"][0] == 1
    sess.step_lagged([0], obs[1], avail, one(0.5, np.float32), one(0, np.uint8), 0.0)
    assert sess.pos[0] == 2 and sess.ring["reward"][0, 0] == 0.5 and sess.ring["done"][0, 0] == 0
    _, tr = sess.step_lagged([0], obs[2], avail, one(-2.0, np.float32), one(1, np.uint8), 0.0, trace=("q",))
    assert sess.slot[0] == 1 and sess.pos[0] == 1 and sess.ep_count[0] == 1
    assert list(sess.ring["reward"][0]) == [0.5, -2.0, 0.0] and list(sess.ring["done"][0]) == [0, 1, 0]
    assert sess.ring["slot_len"][0] == 2 and sess.ring["slot_complete"][0] == 1 and sess.ring["slot_complete"][1] == 0
    assert sess.ring["slot_epid"][1] == 1 and sess.counters[oracle.CNT_EPISODES] == 1
    for i in range(n):
        q0, _ = oracle.agent_forward(cfg, w, obs[2, 0, i], i, -1, np.zeros(H, np.float32))
        assert np.array_equal(tr["q"][0, i], q0)
    # two more records fill the slot (length 3); the next call truncates it
    sess.step_lagged([0], obs[3], avail, one(1.0, np.float32), one(0, np.uint8), 0.0)
    sess.step_lagged([0], obs[4], avail, one(2.0, np.float32), one(0, np.uint8), 0.0)
    assert sess.pos[0] == 3 and sess.ring["slot_len"][1] == 3 and sess.ring["slot_complete"][1] == 0
    sess.step_lagged([0], obs[0], avail, one(3.0, np.float32), one(0, np.uint8), 0.0)
    assert sess.slot[0] == 0 and sess.pos[0] == 1 and sess.ep_count[0] == 2
    assert list(sess.ring["reward"][1]) == [1.0, 2.0, 3.0] and sess.ring["slot_complete"][1] == 1
    assert sess.counters[oracle.CNT_TRUNCATED] == 1 and sess.ring["slot_epid"][0] == 2

"""The step over a list of environments (asynchronous actors, Sec. III-A): the CUDA library against the oracle,
call by call, on seeded environment lists of changing size and order."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_05248_b200 import binding, workloads
from referee import RTOL, check_near_ties, near_tie_rows_allowed, row_rel_err, sample_env_tiles

pytestmark = pytest.mark.gpu


def _env_block(cfg, T):
    E = cfg["E"]
    obs = np.zeros((T, E, cfg["n"], cfg["D"]), np.float32)
    avail = np.zeros((T, E, cfg["n"], cfg["A"]), np.uint8)
    rew = np.zeros((T, E), np.float32)
    done = np.zeros((T, E), np.uint8)
    for t in range(T):
        for e in range(E):
            obs[t, e], avail[t, e], rew[t, e], done[t, e] = oracle.env_emit(cfg, cfg["env"], t, e)
    return obs, avail, rew, done


@pytest.mark.parametrize("prec,kernel,shape,full_every", [
    ("fp32", "ffma", dict(E=96, n=4, A=7, D=24, C=192), 0),
    ("bf16", "ffma", dict(E=700, n=5, A=11, D=13, C=700), 0),
    ("fp32", "ffma", dict(E=3, n=3, A=9, D=30, C=6), 4),
    # the pipelined tensor-core kernel: bulk-copied rows; several tiles with a ragged last one and partial chunks
    ("bf16", "pipelined", dict(E=96, n=4, A=8, D=24, C=192), 5),
    ("bf16", "pipelined", dict(E=700, n=8, A=14, D=80, C=700), 0),
    # rows that are not 16-byte multiples: lists whose length is not a multiple of four go to the CUDA-core kernel
    ("bf16", "pipelined", dict(E=300, n=5, A=12, D=55, C=300), 6)])
def test_subset_steps_match_the_oracle(prec, kernel, shape, full_every):
    cfg = workloads.small_config(H=64, L=5, T=22, precision=prec, env=dict(done_thresh24=1 << 21), **shape)
    E, n, A, T = cfg["E"], cfg["n"], cfg["A"], cfg["T"]
    w = workloads.make_weights(cfg)
    obs, avail, rew, done = _env_block(cfg, T)
    dev = "cuda:0"
    d_obs, d_avail, d_rew, d_done = (torch.as_tensor(x, device=dev) for x in (obs, avail, rew, done))
    actor = binding.Actor(cfg, device=dev, kernel=kernel)
    actor.set_weights(w)
    assert actor.kernel_name == {"ffma": "ffma", "pipelined": "tcgen05-pipelined"}[kernel]
    g_acts, g_q = actor.set_trace(T, want_q=True)
    sess = oracle.Session(cfg, w, np.arange(E))
    rng = np.random.default_rng(7)
    eps, rtol = 0.15, RTOL[prec]
    near = greedy = 0
    for t in range(T):
        if full_every and t % full_every == full_every - 1:
            ids = np.arange(E)
            act = actor.step(d_obs[t], d_avail[t], d_rew[t], d_done[t], eps)
        else:
            M = int(rng.integers(1, E + 1)) if t % 3 else E          # every third call lists everybody, shuffled
            ids = rng.permutation(E)[:M].astype(np.int32)
            tid = torch.as_tensor(ids, device=dev, dtype=torch.long)
            act = actor.step_subset(ids, d_obs[t].index_select(0, tid).contiguous(),
                                    d_avail[t].index_select(0, tid).contiguous(), d_rew[t].index_select(0, tid).contiguous(),
                                    d_done[t].index_select(0, tid).contiguous(), eps)
        act = act.cpu().numpy()
        tid = torch.as_tensor(ids, device=dev, dtype=torch.long)
        q_rows = g_q[t].index_select(0, tid).cpu().numpy()
        assert np.array_equal(g_acts[t].index_select(0, tid).cpu().numpy(), act)
        o_act, tr = sess.step_subset(ids, obs[t, ids], avail[t, ids], rew[t, ids], done[t, ids], eps, adopt=act,
                                     trace=("q", "action_free", "explore"))
        # the decision follows from the library's own Q row, the mask and the draw keyed by the environment's index
        N = len(ids) * n
        re_act, re_ex = oracle.select_batch(q_rows.reshape(N, A), avail[t, ids].reshape(N, A), np.float32(eps),
                                            cfg["seed"], np.uint32(t), np.repeat(ids.astype(np.uint32), n),
                                            np.tile(np.arange(n, dtype=np.uint32), len(ids)))
        assert np.array_equal(re_act, act.reshape(N)), f"call {t}"
        assert np.array_equal(re_ex, tr["explore"].reshape(N))
        assert row_rel_err(q_rows, tr["q"]).max() <= rtol, f"call {t}"
        diff = np.argwhere(tr["action_free"][None] != act[None])
        check_near_ties(diff, tr["q"][None], q_rows[None], tr["action_free"][None], act[None], tr["explore"][None])
        near += len(diff)
        greedy += int((tr["explore"] == 0).sum())
        # rows of the trace that were not listed keep the trace's fill value
        if len(ids) < E:
            rest = torch.as_tensor(np.setdiff1d(np.arange(E), ids), device=dev, dtype=torch.long)
            assert bool((g_acts[t].index_select(0, rest) == -7).all())
    assert near <= near_tie_rows_allowed(prec, greedy), (near, greedy)
    torch.cuda.synchronize()
    st = actor.get_state()
    for k in ("last_action", "slot", "pos", "ep_count"):
        assert np.array_equal(st[k].cpu().numpy(), getattr(sess, k)), k
    assert row_rel_err(st["h"].cpu().numpy(), sess.h).max() <= rtol
    assert st["step"] == T
    rv = actor.ring_view()
    for k in ("slot_epid", "slot_len", "slot_complete"):
        assert np.array_equal(rv[k].cpu().numpy(), sess.ring[k]), k
    written = np.arange(cfg["L"])[None, :] < sess.ring["slot_len"][:, None]
    assert written.sum() > 0
    for k in ("obs", "avail", "action", "reward", "done"):
        assert np.array_equal(rv[k].cpu().numpy()[written], sess.ring[k][written]), k
    assert row_rel_err(rv["q"].cpu().numpy()[written], sess.ring["q"][written]).max() <= rtol
    status, counters = actor.status()
    assert status == 0
    oc = sess.counters
    assert counters["agent_steps"] == oc[oracle.CNT_STEPS] and counters["episodes"] == oc[oracle.CNT_EPISODES]
    assert counters["explored"] == oc[oracle.CNT_EXPLORE] and counters["truncated"] == oc[oracle.CNT_TRUNCATED]
    assert counters["episodes"] > 0
    actor.destroy()


def test_subset_list_is_validated_on_the_host():
    cfg = workloads.small_config(H=64, D=8, E=16, C=32, L=4, T=4, precision="fp32", n=2, A=4)
    actor = binding.Actor(cfg)
    actor.set_weights(workloads.make_weights(cfg))
    z = lambda *s, dt=torch.float32: torch.zeros(s, dtype=dt, device="cuda:0")
    def call(ids):
        M = len(ids)
        return actor.step_subset(np.array(ids, np.int32), z(M, 2, 8), torch.ones((M, 2, 4), dtype=torch.uint8, device="cuda:0"),
                                 z(M), z(M, dt=torch.uint8), 0.0)
    launches = actor.launch_count
    for bad in ([3, 3], [0, 16], [-1], list(range(16)) + [0]):
        with pytest.raises(binding.MarlError):
            call(bad)
    assert actor.get_state()["step"] == 0 and actor.launch_count == launches
    call([5, 2])
    assert actor.get_state()["step"] == 1
    st = actor.get_state()
    assert sorted(torch.nonzero(st["pos"]).flatten().tolist()) == [2, 5]
    actor.destroy()


@pytest.mark.parametrize("prec,kernel,shape", [("fp32", "ffma", dict(E=80, n=3, A=6, D=20, C=240)),
                                               ("bf16", "ffma", dict(E=500, n=5, A=11, D=16, C=1000)),
                                               ("bf16", "pipelined", dict(E=64, n=4, A=8, D=24, C=128)),
                                               ("bf16", "pipelined", dict(E=700, n=8, A=14, D=80, C=1400)),
                                               ("bf16", "pipelined", dict(E=300, n=5, A=12, D=55, C=600))])
def test_lagged_steps_match_the_oracle(prec, kernel, shape):
    """Environments that answer after the action (Algorithm 1): every environment runs on its own clock, a call lists
    those with a new observation and brings the outcome of their previous action."""
    cfg = workloads.small_config(H=64, L=4, T=26, precision=prec, env=dict(done_thresh24=1 << 22), **shape)
    E, n, A, T = cfg["E"], cfg["n"], cfg["A"], cfg["T"]
    w = workloads.make_weights(cfg)
    obs, avail, rew, done = _env_block(cfg, T)            # [k][e]: the k-th exchange of environment e
    dev = "cuda:0"
    actor = binding.Actor(cfg, device=dev, kernel=kernel)
    actor.set_weights(w)
    g_acts, g_q = actor.set_trace(T, want_q=True)
    sess = oracle.Session(cfg, w, np.arange(E))
    rng = np.random.default_rng(11)
    k_of = np.zeros(E, np.int64)                          # exchanges each environment has had
    eps, rtol = 0.1, RTOL[prec]
    near = greedy = 0
    for t in range(T):
        M = E if t == 0 else int(rng.integers(1, E + 1))
        ids = rng.permutation(E)[:M].astype(np.int32)
        k = k_of[ids]
        first = k == 0
        p_rew = np.where(first, np.float32(7.0), rew[np.maximum(k - 1, 0), ids]).astype(np.float32)
        p_done = np.where(first, 1, done[np.maximum(k - 1, 0), ids]).astype(np.uint8)   # ignored on a first call
        o, av = obs[k, ids], avail[k, ids]
        act = actor.step_lagged(ids, *(torch.as_tensor(x, device=dev) for x in (o, av, p_rew, p_done)), eps).cpu().numpy()
        tid = torch.as_tensor(ids, device=dev, dtype=torch.long)
        q_rows = g_q[t].index_select(0, tid).cpu().numpy()
        _, tr = sess.step_lagged(ids, o, av, p_rew, p_done, eps, adopt=act, trace=("q", "action_free", "explore"))
        N = M * n
        re_act, re_ex = oracle.select_batch(q_rows.reshape(N, A), av.reshape(N, A), np.float32(eps), cfg["seed"],
                                            np.uint32(t), np.repeat(ids.astype(np.uint32), n),
                                            np.tile(np.arange(n, dtype=np.uint32), M))
        assert np.array_equal(re_act, act.reshape(N)), f"call {t}"
        assert np.array_equal(re_ex, tr["explore"].reshape(N))
        assert row_rel_err(q_rows, tr["q"]).max() <= rtol, f"call {t}"
        diff = np.argwhere(tr["action_free"][None] != act[None])
        check_near_ties(diff, tr["q"][None], q_rows[None], tr["action_free"][None], act[None], tr["explore"][None])
        near += len(diff)
        greedy += int((tr["explore"] == 0).sum())
        k_of[ids] += 1
    assert near <= near_tie_rows_allowed(prec, greedy), (near, greedy)
    torch.cuda.synchronize()
    st = actor.get_state()
    for key in ("last_action", "slot", "pos", "ep_count"):
        assert np.array_equal(st[key].cpu().numpy(), getattr(sess, key)), key
    assert row_rel_err(st["h"].cpu().numpy(), sess.h).max() <= rtol
    rv = actor.ring_view()
    for key in ("slot_epid", "slot_len", "slot_complete"):
        assert np.array_equal(rv[key].cpu().numpy(), sess.ring[key]), key
    written = np.arange(cfg["L"])[None, :] < sess.ring["slot_len"][:, None]
    for key in ("obs", "avail", "action", "reward", "done"):
        assert np.array_equal(rv[key].cpu().numpy()[written], sess.ring[key][written]), key
    assert row_rel_err(rv["q"].cpu().numpy()[written], sess.ring["q"][written]).max() <= rtol
    status, counters = actor.status()
    oc = sess.counters
    assert status == 0 and counters["agent_steps"] == oc[oracle.CNT_STEPS]
    assert counters["episodes"] == oc[oracle.CNT_EPISODES] > 0 and counters["truncated"] == oc[oracle.CNT_TRUNCATED] > 0
    actor.destroy()


@pytest.mark.parametrize("lagged", [False, True])
def test_list_steps_full_size_bench_configuration(lagged):
    """The workload and launch configuration that `bench.py --subset 0.5 [--lagged]` times (E=65536, lists of 32768
    environments, 20 GB ring, pipelined tensor-core kernel in list mode): the oracle recomputes 4096 environments
    (seeded whole tiles), each on its own clock, through every call that lists it."""
    cfg = workloads.config(5)
    E, n, A, D = cfg["E"], cfg["n"], cfg["A"], cfg["D"]
    calls, M, eps = 6, E // 2, 0.05
    w = workloads.make_weights(cfg)
    dev = "cuda:0"
    actor = binding.Actor(cfg, device=dev, kernel="auto", work_steps=1)
    assert actor.kernel_name == "tcgen05-pipelined"
    actor.set_weights(w)
    g_acts, g_q = actor.set_trace(calls, want_q=True)
    staged = actor.env_generate(cfg["env"], 0, calls)                    # [k][e]: the k-th exchange of environment e
    sample = sample_env_tiles(E, 128 // n, 4096, seed=9)                  # whole tiles of the dense order
    where = {int(e): x for x, e in enumerate(sample)}
    o_obs, o_avail = np.zeros((calls, len(sample), n, D), np.float32), np.zeros((calls, len(sample), n, A), np.uint8)
    o_rew, o_done = np.zeros((calls, len(sample)), np.float32), np.zeros((calls, len(sample)), np.uint8)
    for k in range(calls):
        for x, e in enumerate(sample):
            o_obs[k, x], o_avail[k, x], o_rew[k, x], o_done[k, x] = oracle.env_emit(cfg, cfg["env"], k, int(e))
    sess = oracle.Session(cfg, w, sample)
    rng = np.random.default_rng(3)
    k_of = np.zeros(E, np.int64)
    rtol = RTOL[cfg["precision"]]
    rows = near = listed = greedy = 0
    for t in range(calls):
        ids = rng.permutation(E)[:M].astype(np.int32)
        if t % 2 == 0:                                                    # the sample is listed often
            ids[: len(sample)] = rng.permutation(sample)
        ids = np.array(list(dict.fromkeys(ids.tolist())), np.int32)       # no environment twice
        ids = ids[: len(ids) // 4 * 4]
        listed += len(ids)
        tid = torch.as_tensor(ids, device=dev, dtype=torch.long)
        k = torch.as_tensor(k_of[ids], device=dev)
        km1 = torch.clamp(k - 1, min=0)
        if lagged:
            rew = torch.where(k > 0, staged[2][km1, tid], torch.zeros_like(staged[2][0, tid]))
            done = torch.where(k > 0, staged[3][km1, tid], torch.zeros_like(staged[3][0, tid]))
            act = actor.step_lagged(ids, staged[0][k, tid].contiguous(), staged[1][k, tid].contiguous(), rew.contiguous(),
                                    done.contiguous(), eps)
        else:
            act = actor.step_subset(ids, staged[0][k, tid].contiguous(), staged[1][k, tid].contiguous(),
                                    staged[2][k, tid].contiguous(), staged[3][k, tid].contiguous(), eps)
        pick = np.nonzero(np.isin(ids, sample))[0]                        # rows of the call that the oracle follows
        s_ids = ids[pick]
        sx = np.array([where[int(e)] for e in s_ids])
        ks = k_of[s_ids]
        act_s = act[torch.as_tensor(pick, device=dev)].cpu().numpy()
        q_s = g_q[t].index_select(0, torch.as_tensor(s_ids, device=dev, dtype=torch.long)).cpu().numpy()
        if lagged:
            p_r = np.where(ks > 0, o_rew[np.maximum(ks - 1, 0), sx], 0).astype(np.float32)
            p_d = np.where(ks > 0, o_done[np.maximum(ks - 1, 0), sx], 0).astype(np.uint8)
            _, tr = sess.step_lagged(s_ids, o_obs[ks, sx], o_avail[ks, sx], p_r, p_d, eps, adopt=act_s,
                                     trace=("q", "action_free", "explore"))
        else:
            _, tr = sess.step_subset(s_ids, o_obs[ks, sx], o_avail[ks, sx], o_rew[ks, sx], o_done[ks, sx], eps, adopt=act_s,
                                     trace=("q", "action_free", "explore"))
        N = len(s_ids) * n
        re_act, _ = oracle.select_batch(q_s.reshape(N, A), o_avail[ks, sx].reshape(N, A), np.float32(eps), cfg["seed"],
                                        np.uint32(t), np.repeat(s_ids.astype(np.uint32), n),
                                        np.tile(np.arange(n, dtype=np.uint32), len(s_ids)))
        assert np.array_equal(re_act, act_s.reshape(N)), f"call {t}"
        assert row_rel_err(q_s, tr["q"]).max() <= rtol, f"call {t}"
        diff = np.argwhere(tr["action_free"][None] != act_s[None])
        check_near_ties(diff, tr["q"][None], q_s[None], tr["action_free"][None], act_s[None], tr["explore"][None])
        near += len(diff)
        greedy += int((tr["explore"] == 0).sum())
        rows += N
        # the whole call: every chosen action is available
        chosen = torch.gather(staged[1][k, tid], 2, act.unsqueeze(-1).long()).squeeze(-1)
        assert bool((chosen == 1).all())
        k_of[ids] += 1
    assert rows >= 4096 * n * 3 and near <= near_tie_rows_allowed(cfg["precision"], greedy), (near, greedy)
    torch.cuda.synchronize()
    st = actor.get_state()
    ts = torch.as_tensor(sample, device=dev, dtype=torch.long)
    for key in ("last_action", "slot", "pos", "ep_count"):
        assert np.array_equal(st[key].index_select(0, ts).cpu().numpy(), getattr(sess, key)), key
    assert row_rel_err(st["h"].index_select(0, ts).cpu().numpy(), sess.h).max() <= rtol
    rv = actor.ring_view()
    S = sess.S
    slots = torch.as_tensor((sample[:, None] * S + np.arange(S)[None, :]).reshape(-1), device=dev, dtype=torch.long)
    for key in ("slot_epid", "slot_len", "slot_complete"):
        assert np.array_equal(rv[key].index_select(0, slots).cpu().numpy(), sess.ring[key]), key
    written = np.arange(cfg["L"])[None, :] < sess.ring["slot_len"][:, None]
    for key in ("obs", "avail", "action", "reward", "done"):
        assert np.array_equal(rv[key].index_select(0, slots).cpu().numpy()[written], sess.ring[key][written]), key
    status, counters = actor.status()
    assert status == 0 and counters["agent_steps"] == listed * n
    del staged, g_acts, g_q
    actor.destroy()

"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2205_05248_b200 import binding, workloads
from referee import RTOL, referee, row_rel_err, run_gpu_rollout, sample_env_tiles, sample_envs

pytestmark = pytest.mark.gpu


def _oracle_env_block(cfg, ids, t0, n_steps):
    obs = np.zeros((n_steps, len(ids), cfg["n"], cfg["D"]), np.float32)
    avail = np.zeros((n_steps, len(ids), cfg["n"], cfg["A"]), np.uint8)
    rew = np.zeros((n_steps, len(ids)), np.float32)
    done = np.zeros((n_steps, len(ids)), np.uint8)
    for s in range(n_steps):
        for x, e in enumerate(ids):
            obs[s, x], avail[s, x], rew[s, x], done[s, x] = oracle.env_emit(cfg, cfg["env"], t0 + s, int(e))
    return obs, avail, rew, done


@pytest.mark.parametrize("k,t0,n_steps,n_ids", [(1, 0, 16, 8), (2, 5, 3, 24), (3, 250, 2, 24), (4, 77, 2, 24),
                                                (5, 63, 1, 16)])
def test_env_generate_bit_exact(k, t0, n_steps, n_ids):
    """Every synthetic-environment stream equals the oracle's, bit for bit, at the full batch size."""
    cfg = workloads.config(k, E=4096) if k == 5 else workloads.config(k)
    actor = binding.Actor(cfg, kernel="ffma", work_steps=1)
    obs, avail, rew, done = actor.env_generate(cfg["env"], t0, n_steps)
    ids = sample_envs(cfg["E"], n_ids, seed=k)
    t = torch.as_tensor(ids, device=obs.device)
    o_obs, o_avail, o_rew, o_done = _oracle_env_block(cfg, ids, t0, n_steps)
    assert np.array_equal(obs.index_select(1, t).cpu().numpy().view(np.uint32), o_obs.view(np.uint32))
    assert np.array_equal(avail.index_select(1, t).cpu().numpy(), o_avail)
    assert np.array_equal(rew.index_select(1, t).cpu().numpy().view(np.uint32), o_rew.view(np.uint32))
    assert np.array_equal(done.index_select(1, t).cpu().numpy(), o_done)
    # whole-batch properties that hold at any size
    assert bool((avail[..., 0] == 1).all())
    assert float(obs.abs().max()) <= 3.0
    actor.destroy()


def test_config1_full_parity_fp32():
    """Workload 1 (3 agents, fp32): every row of every step, no near-tie allowed."""
    cfg = workloads.config(1)
    w = workloads.make_weights(cfg)
    actor, acts, q = run_gpu_rollout(cfg, w)
    res = referee(cfg, w, actor, acts, q, near_tie_budget=0.0)
    assert res["rows"] == 384 and res["kernel"] == "ffma"
    actor.destroy()


@pytest.mark.parametrize("k,n_ids", [(2, None), (3, None), (4, 4096)])
def test_configs_2_to_4_parity(k, n_ids):
    """Full-size GPU rollout; the oracle recomputes every environment of workloads 2 and 3, and for workload 4
    whole tiles (the first, the last, and seeded ones from every wave of the launch) adding up to 4096."""
    cfg = workloads.config(k)
    w = workloads.make_weights(cfg)
    actor, acts, q = run_gpu_rollout(cfg, w)
    ids = None if n_ids is None else sample_env_tiles(cfg["E"], 128 // cfg["n"] // 4 * 4, n_ids, seed=k)
    res = referee(cfg, w, actor, acts, q, env_ids=ids)
    assert res["envs"] >= min(cfg["E"], 4096)
    print(f"cfg{k}: {res}")
    # properties over the whole batch: every chosen action is available; every step was recorded
    rv = actor.ring_view()
    status, counters = actor.status()
    assert status == 0 and counters["agent_steps"] == cfg["E"] * cfg["n"] * cfg["T"]
    lens = rv["slot_len"].cpu().numpy()
    assert lens.max() <= cfg["L"]
    actor.destroy()


@pytest.mark.parametrize("H,prec,kernel", [(64, "bf16", "auto"), (64, "bf16", "dual"), (64, "bf16", "tensor"), (64, "bf16", "ffma"),
                                           (128, "bf16", "auto"), (128, "bf16", "ffma"), (64, "fp32", "ffma"),
                                           (128, "fp32", "ffma")])
def test_config5_parity_small_E(H, prec, kernel):
    cfg = workloads.config(5, E=4096, H=H, precision=prec)
    cfg["T"] = 24
    w = workloads.make_weights(cfg)
    actor, acts, q = run_gpu_rollout(cfg, w, kernel=kernel)
    if kernel == "auto":
        assert actor.kernel_name == ("tcgen05-streamed" if H == 128 else "tcgen05-pipelined")
    res = referee(cfg, w, actor, acts, q)          # every environment
    print(f"cfg5 H={H} {prec} {kernel}: {res}")
    actor.destroy()


def test_config5_full_size_bench_configuration():
    """The workload and launch configuration that bench.py times (E=65536, H=64, bf16, T=64, 20 GB ring, tcgen05
    kernel, one marl_rollout_staged call on pre-staged inputs); the oracle recomputes a seeded subset of
    environments (4096 of them, in whole tiles), and whole-batch properties are checked on everything."""
    cfg = workloads.config(5)
    w = workloads.make_weights(cfg)
    actor = binding.Actor(cfg, kernel="auto", work_steps=1)
    assert actor.kernel_name == "tcgen05-pipelined"
    actor.set_weights(w)
    acts, q = actor.set_trace(cfg["T"])
    staged = actor.env_generate(cfg["env"], 0, cfg["T"])
    actor.rollout_staged(*staged, cfg["T"], cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    torch.cuda.synchronize()
    ids = sample_env_tiles(cfg["E"], 128 // cfg["n"], 4096, seed=5)   # 256 whole tiles over all 28 waves
    assert len(ids) >= 4096 and ids[0] == 0 and ids[-1] == cfg["E"] - 1
    res = referee(cfg, w, actor, acts, q, env_ids=ids)
    print(f"cfg5 full size: {res}")
    status, counters = actor.status()
    assert status == 0 and counters["agent_steps"] == cfg["E"] * cfg["n"] * cfg["T"]
    # every chosen action is available, in every row of every step
    avail = staged[1]
    chosen = torch.gather(avail, 3, acts[: cfg["T"]].unsqueeze(-1).long()).squeeze(-1)
    assert bool((chosen == 1).all())
    # explore share ~ eps over 33.5 M rows
    assert abs(counters["explored"] / counters["agent_steps"] - cfg["eps_start"]) < 1e-3
    # slot headers against the done stream (one slot per environment here, so a new episode reuses the slot)
    rv = actor.ring_view()
    done = staged[3].long()                                            # [T][E]
    T = cfg["T"]
    idx = torch.arange(T, device=done.device)[:, None] * done          # step index where done, else 0
    last_done = torch.where(done.any(0), idx.max(0).values, torch.full_like(idx[0], -1))
    before = torch.where(idx < last_done[None, :], idx, torch.zeros_like(idx))   # done steps before the last one
    prev_done = torch.where((done.sum(0) > 1), before.max(0).values, torch.full_like(last_done, -1))
    closed_now = last_done == T - 1
    want_len = torch.where(closed_now, last_done - prev_done, (T - 1) - last_done)
    want_len = torch.where(want_len == 0, torch.ones_like(want_len), want_len)
    got_len = rv["slot_len"].long()
    open_or_closed = torch.where(closed_now, rv["slot_complete"].long() == 1, rv["slot_complete"].long() == 0)
    assert bool(open_or_closed.all())
    assert bool((got_len[~closed_now] == ((T - 1) - last_done)[~closed_now]).all())
    assert bool((got_len[closed_now] == want_len[closed_now]).all())
    del staged, acts, q
    actor.destroy()


def test_ragged_tiles_and_tiny_shapes():
    """Tile tails (E not a multiple of the tile), one agent, one action, one environment."""
    for over in (dict(E=37, n=5, C=74), dict(E=1, n=1, A=1, C=2), dict(E=150, n=7, A=32, D=3, C=150),
                 dict(E=9, n=32, A=2, D=17, C=9), dict(E=300, n=3, D=129, C=300)):
        cfg = workloads.small_config(H=64, L=7, T=20, **over)
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel="ffma")
        referee(cfg, w, actor, acts, q)
        actor.destroy()


def test_tensor_kernel_ragged_tiles_and_tiny_shapes():
    """The tcgen05 kernel on tile tails, agent counts that do not divide 128, one row, 32 actions."""
    for over in (dict(E=37, n=5, D=16, C=74), dict(E=1, n=1, A=1, D=8, C=2), dict(E=150, n=7, A=32, D=24, C=150),
                 dict(E=9, n=32, A=2, D=40, C=9), dict(E=300, n=3, D=96, C=300), dict(E=130, n=8, D=80, A=14, C=260)):
        cfg = workloads.small_config(H=64, L=7, T=20, precision="bf16", **over)
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel="tensor")
        res = referee(cfg, w, actor, acts, q)
        assert res["kernel"] == "tcgen05"
        actor.destroy()


def _assert_same_rollout(a, acts_a, q_a, b, acts_b, q_b, tag=""):
    """Two kernels that run the same arithmetic (the Q accumulation starts from the bias in one and ends with it in
    the other, so Q may differ in the last bits): identical decisions, records, headers and state."""
    assert torch.equal(acts_a, acts_b), tag
    assert torch.allclose(q_a, q_b, rtol=1e-4, atol=2e-6), tag
    ra, rb = a.ring_view(), b.ring_view()
    for k in ("obs", "avail", "action", "reward", "done", "slot_epid", "slot_len", "slot_complete"):
        assert torch.equal(ra[k], rb[k]), (tag, k)
    assert torch.allclose(ra["q"], rb["q"], rtol=1e-4, atol=2e-6), tag
    sa, sb = a.get_state(), b.get_state()
    for key in ("last_action", "slot", "pos", "ep_count"):
        assert torch.equal(sa[key], sb[key]), (tag, key)
    assert torch.allclose(sa["h"], sb["h"], rtol=1e-4, atol=2e-6), tag
    assert a.status() == b.status(), tag


def test_pipelined_tensor_kernel_ragged_tiles_and_shapes():
    """The pipelined tcgen05 kernel on tile tails, partial staging chunks (environment counts that are not
    multiples of four), one tile, fewer tiles than blocks and more, agent counts that do not divide 128,
    32 actions, observation widths that need padding to the MMA's K step."""
    for over in (dict(E=130, n=8, D=80, A=14, C=260), dict(E=1, n=4, A=4, D=8, C=2), dict(E=37, n=16, A=5, D=16, C=74),
                 dict(E=150, n=7, A=32, D=24, C=150), dict(E=9, n=32, A=2, D=40, C=9), dict(E=2500, n=8, A=6, D=72, C=2500),
                 dict(E=333, n=5, A=16, D=88, C=333),
                 # shapes whose per-environment blocks are not 16-byte multiples (word-by-word converter path)
                 dict(E=36, n=5, A=12, D=55, C=72), dict(E=8, n=6, A=6, D=13, C=16), dict(E=300, n=4, A=5, D=30, C=300)):
        cfg = workloads.small_config(H=64, L=7, T=20, precision="bf16", **over)
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel="pipelined")
        assert actor.kernel_name == "tcgen05-pipelined"
        # the one-tile kernel does the same arithmetic: same decisions, same records
        try:
            one, acts1, q1 = run_gpu_rollout(cfg, w, kernel="tensor")
        except binding.MarlError:      # a shape the one-tile kernel does not take (record buffers too large, D % 8)
            one = None
            assert over["D"] in (88, 55, 13, 30)
        if one is not None:
            _assert_same_rollout(actor, acts, q, one, acts1, q1, tag=str(over))
            one.destroy()
        referee(cfg, w, actor, acts, q)
        actor.destroy()


def test_pipelined_and_one_tile_kernels_write_the_same_ring():
    """Both tensor-core kernels run the same arithmetic: identical actions, records, headers and state (Q and h to
    the last bits)."""
    cfg = workloads.config(2, E=600)
    cfg["T"] = 40
    w = workloads.make_weights(cfg)
    a, acts_a, q_a = run_gpu_rollout(cfg, w, kernel="pipelined")
    b, acts_b, q_b = run_gpu_rollout(cfg, w, kernel="tensor")
    assert a.kernel_name == "tcgen05-pipelined" and b.kernel_name == "tcgen05"
    _assert_same_rollout(a, acts_a, q_a, b, acts_b, q_b)
    a.destroy()
    b.destroy()


@pytest.mark.parametrize("kernel,prec,shape", [("ffma", "fp32", {}), ("tensor", "bf16", {}),
                                               ("pipelined", "bf16", dict(n=4, A=8))])
def test_done_every_step_and_never(kernel, prec, shape):
    for thr, L in ((1 << 24, 4), (0, 5)):
        cfg = workloads.small_config(H=64, D=8, E=40, C=80, L=L, T=17, precision=prec, env=dict(done_thresh24=thr),
                                     **shape)
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel=kernel)
        res = referee(cfg, w, actor, acts, q)
        _, counters = actor.status()
        if thr:
            assert counters["episodes"] == 40 * 17 and counters["truncated"] == 0
        else:
            assert counters["truncated"] == counters["episodes"] == 40 * (17 // 5)
        actor.destroy()


@pytest.mark.parametrize("kernel,prec,shape", [("ffma", "fp32", {}), ("tensor", "bf16", {}),
                                               ("pipelined", "bf16", dict(n=8, A=6))])
def test_annealed_epsilon_and_split_rollouts_resume(kernel, prec, shape):
    """eps schedule follows the global step; rollout(T) == rollout(a) + rollout(b); a checkpoint restored
    into a fresh handle continues identically."""
    cfg = workloads.small_config(H=64, D=16, E=64, C=128, L=9, T=30, eps_start=1.0, eps_end=0.05, anneal_steps=29,
                                 precision=prec, **shape)
    w = workloads.make_weights(cfg)
    one, a1, q1 = run_gpu_rollout(cfg, w, kernel=kernel)
    referee(cfg, w, one, a1, q1)
    two, a2, q2 = run_gpu_rollout(cfg, w, kernel=kernel, splits=[11, 19])
    assert torch.equal(a1, a2) and torch.equal(q1, q2)
    r1, r2 = one.ring_view(), two.ring_view()
    assert torch.equal(one.ring_mem, two.ring_mem)
    # checkpoint after 11 steps -> fresh handle -> 19 more
    first = binding.Actor(cfg, kernel=kernel)
    first.set_weights(w)
    first.rollout(cfg["env"], 11, 1.0, 0.05, 29)
    st = first.get_state()
    second = binding.Actor(cfg, kernel=kernel)
    second.set_weights(w)
    second.ring_mem.copy_(first.ring_mem)
    second.set_state(st)
    second.rollout(cfg["env"], 19, 1.0, 0.05, 29)
    torch.cuda.synchronize()
    assert torch.equal(second.ring_mem, one.ring_mem)
    s1, s2 = one.get_state(), second.get_state()
    for key in ("h", "last_action", "slot", "pos", "ep_count"):
        assert torch.equal(s1[key], s2[key]), key
    assert s1["step"] == s2["step"] == 30
    for a in (one, two, first, second):
        a.destroy()


@pytest.mark.parametrize("kernel,prec,A", [("ffma", "fp32", 5), ("tensor", "bf16", 5), ("pipelined", "bf16", 12)])
def test_step_api_equals_rollout_and_host_variant(kernel, prec, A):
    """T calls of marl_actor_step (device inputs) and of marl_actor_step_host (host inputs) reproduce
    marl_rollout: same actions, same ring, same state."""
    cfg = workloads.small_config(H=64, D=24, E=50, n=4, A=A, C=100, L=8, T=12, precision=prec)
    w = workloads.make_weights(cfg)
    ref, acts, q = run_gpu_rollout(cfg, w, kernel=kernel)
    assert ref.kernel_name == {"ffma": "ffma", "tensor": "tcgen05", "pipelined": "tcgen05-pipelined"}[kernel]
    obs, avail, rew, done = ref.env_generate(cfg["env"], 0, cfg["T"])
    dev = binding.Actor(cfg, kernel=kernel)
    dev.set_weights(w)
    host = binding.Actor(cfg, kernel=kernel)
    host.set_weights(w)
    h_obs, h_avail, h_rew, h_done = [t.cpu().pin_memory() for t in (obs, avail, rew, done)]
    h_act = torch.empty((cfg["E"], cfg["n"]), dtype=torch.int32).pin_memory()
    for t in range(cfg["T"]):
        a = dev.step(obs[t], avail[t], rew[t], done[t], cfg["eps_start"])
        assert torch.equal(a, acts[t])
        host.step_host(h_obs[t], h_avail[t], h_rew[t], h_done[t], cfg["eps_start"], h_act)
        assert torch.equal(h_act, acts[t].cpu())
    torch.cuda.synchronize()
    assert torch.equal(dev.ring_mem, ref.ring_mem) and torch.equal(host.ring_mem, ref.ring_mem)
    for key in ("h", "last_action", "slot", "pos", "ep_count"):
        assert torch.equal(dev.get_state()[key], ref.get_state()[key]), key
    for a in (ref, dev, host):
        a.destroy()


def test_determinism_same_seed_same_bytes():
    cfg = workloads.config(2, E=512)
    cfg["T"] = 16
    w = workloads.make_weights(cfg)
    a, acts_a, q_a = run_gpu_rollout(cfg, w)
    b, acts_b, q_b = run_gpu_rollout(cfg, w)
    assert torch.equal(acts_a, acts_b) and torch.equal(q_a, q_b)
    ra, rb = a.ring_view(), b.ring_view()
    for k in ("obs", "avail", "action", "q", "reward", "done", "slot_epid", "slot_len", "slot_complete"):
        assert torch.equal(ra[k], rb[k]), k
    a.destroy()
    b.destroy()


@pytest.mark.parametrize("kernel,shape", [("ffma", dict(n=2)), ("tensor", dict(n=4, A=8, D=8, precision="bf16")),
                                          ("pipelined", dict(n=4, A=8, D=8, precision="bf16"))])
def test_no_available_action_is_reported_not_fatal(kernel, shape):
    """A row whose mask is all zero takes action 0, sets the status bit and counts it."""
    cfg = workloads.small_config(H=64, E=6, C=6, L=8, T=1, **shape)
    w = workloads.make_weights(cfg)
    actor = binding.Actor(cfg, kernel=kernel)
    actor.set_weights(w)
    obs, avail, rew, done = actor.env_generate(cfg["env"], 0, 1)
    avail[0, 3, 1, :] = 0
    acts = actor.step(obs[0], avail[0], rew[0], done[0], 0.0)
    status, counters = actor.status()
    assert status & binding.STATUS_NO_AVAIL and counters["no_avail"] == 1
    assert int(acts[3, 1]) == 0
    sess = oracle.Session(cfg, w, np.arange(cfg["E"]))
    o_acts, _ = sess.step(obs[0].cpu().numpy(), avail[0].cpu().numpy(), rew[0].cpu().numpy(), done[0].cpu().numpy(), 0.0)
    assert sess.counters[oracle.CNT_NO_AVAIL] == 1 and int(o_acts[3, 1]) == 0
    if kernel == "ffma":                     # (the bf16 kernels may differ from the oracle in a near-tie elsewhere)
        assert np.array_equal(acts.cpu().numpy(), o_acts)
    actor.destroy()


@pytest.mark.parametrize("kernel,shape", [("ffma", {}), ("tensor", dict(n=4, A=8, D=8, precision="bf16")),
                                          ("pipelined", dict(n=4, A=8, D=8, precision="bf16"))])
def test_bad_cursor_sets_status_and_skips(kernel, shape):
    """A corrupted ring cursor handed in through set_state is detected; nothing is written out of range."""
    cfg = workloads.small_config(H=64, E=4, C=4, L=8, T=2, **shape)
    w = workloads.make_weights(cfg)
    actor = binding.Actor(cfg, kernel=kernel)
    actor.set_weights(w)
    st = actor.get_state()
    bad = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in st.items()}
    bad["pos"][2] = 99
    actor.set_state(bad)
    before = actor.ring_mem.clone()
    actor.rollout(cfg["env"], 2, 0.1)
    status, _ = actor.status()
    assert status & binding.STATUS_BAD_INDEX
    rv = actor.ring_view()
    assert int(rv["slot_len"][2]) == 0
    # the records: nothing of the corrupted environment's slot was touched, and of every other slot only the two
    # records that the two steps wrote (one slot per environment here)
    meta = rv["meta"]
    base = meta["base"] - actor.ring_mem.data_ptr()
    recs_now = actor.ring_mem[base: base + cfg["C"] * meta["slot_stride"]].view(cfg["C"], cfg["L"], meta["step_stride"])
    recs_before = before[base: base + cfg["C"] * meta["slot_stride"]].view(cfg["C"], cfg["L"], meta["step_stride"])
    assert torch.equal(recs_now[2], recs_before[2])
    assert torch.equal(recs_now[:, 2:], recs_before[:, 2:])
    for e in (0, 1, 3):
        assert not torch.equal(recs_now[e, :2], recs_before[e, :2])
    actor.destroy()


def test_host_errors_are_codes_not_crashes():
    cfg = workloads.small_config(H=64)
    actor = binding.Actor(cfg, kernel="ffma")
    obs, avail, rew, done = actor.env_generate(cfg["env"], 0, 1)
    with pytest.raises(binding.MarlError, match="set_weights"):
        actor.step(obs[0], avail[0], rew[0], done[0], 0.1)
    actor.set_weights(workloads.make_weights(cfg))
    with pytest.raises(binding.MarlError, match="eps"):
        actor.step(obs[0], avail[0], rew[0], done[0], 1.5)
    with pytest.raises(binding.MarlError):
        actor.rollout(cfg["env"], 0, 0.1)
    actor.destroy()
    with pytest.raises(binding.MarlError, match="tensor-core"):
        binding.Actor(dict(cfg, precision="fp32"), kernel="tensor")


def test_bounded_wait_gives_up_and_context_survives():
    """A device-side wait on a barrier that nothing completes expires, reports TIMEOUT through the status word
    and leaves the context usable (no trap, no hang): the failure path of every hand-off in the tcgen05 kernel."""
    st = binding.marl_selftest_bounded_wait(20000)
    assert st & binding.STATUS_TIMEOUT and st & 0x100
    x = torch.arange(8, device="cuda").sum().item()      # the context still works
    assert x == 28
    for kernel, shape in (("tensor", {}), ("pipelined", dict(n=4, A=8))):
        cfg = workloads.small_config(H=64, D=8, precision="bf16", E=40, C=40, **shape)
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel=kernel)
        assert actor.status()[0] == 0                    # and a real rollout afterwards is clean
        actor.destroy()


def test_pipelined_kernel_falls_back_on_unaligned_inputs():
    """Inputs that are not 16-byte aligned cannot be bulk-copied: a step with unaligned availability bytes runs on
    the one-tile kernel, one with unaligned observations on the FFMA kernel, each with that kernel's exact results;
    the next aligned step is back on the pipelined kernel."""
    cfg = workloads.small_config(H=64, D=24, E=40, n=4, A=12, C=80, L=8, T=3, precision="bf16")
    w = workloads.make_weights(cfg)
    pipe, tens, ffma = (binding.Actor(cfg, kernel=k) for k in ("pipelined", "tensor", "ffma"))
    for a in (pipe, tens, ffma):
        a.set_weights(w)
    obs, avail, rew, done = pipe.env_generate(cfg["env"], 0, 3)

    def shifted(t, elems):                      # a copy that starts `elems` elements into a fresh allocation
        big = torch.empty(t.numel() + 64, dtype=t.dtype, device=t.device)
        out = big[elems:elems + t.numel()].view(t.shape)
        out.copy_(t)
        return out

    # step 0: unaligned availability bytes -> one-tile kernel
    av = shifted(avail[0], 4)
    assert av.data_ptr() % 16 != 0
    a0 = pipe.step(obs[0], av, rew[0], done[0], cfg["eps_start"])
    assert torch.equal(a0, tens.step(obs[0], avail[0], rew[0], done[0], cfg["eps_start"]))
    ffma.step(obs[0], avail[0], rew[0], done[0], cfg["eps_start"])
    # step 1: unaligned observations -> FFMA kernel (from the tensor-core kernels' state: compare decisions only where
    # the hidden states agree to the tolerance, i.e. run the FFMA actor from the same state)
    st = pipe.get_state()
    ffma.set_state(st)
    ffma.ring_mem.copy_(pipe.ring_mem)
    ob = shifted(obs[1], 1)
    assert ob.data_ptr() % 16 != 0
    a1 = pipe.step(ob, avail[1], rew[1], done[1], cfg["eps_start"])
    assert torch.equal(a1, ffma.step(obs[1], avail[1], rew[1], done[1], cfg["eps_start"]))
    torch.cuda.synchronize()
    assert torch.equal(pipe.ring_mem, ffma.ring_mem)
    # step 2: aligned again
    a2 = pipe.step(obs[2], avail[2], rew[2], done[2], cfg["eps_start"])
    assert a2.shape == a1.shape and pipe.status()[0] == 0
    for a in (pipe, tens, ffma):
        a.destroy()


@pytest.mark.parametrize("seed", range(4))
def test_pipelined_kernel_seeded_shapes(seed):
    """Seeded shapes inside the pipelined kernel's stated domain (4..32 agents, 1..32 actions, 1..256 observation
    features; n * A odd or even): environment counts that leave ragged tiles and partial chunks, short and long
    slots, single-step and multi-step launches mixed.  Each is refereed against the oracle on every row."""
    rng = np.random.default_rng(1000 + seed)
    done_shapes = 0
    while done_shapes < 5:
        n = int(rng.integers(4, 33))
        A = int(rng.integers(1, 33))
        D = int(rng.integers(1, 257))
        tile_envs = max(1, 128 // n)
        E = int(rng.integers(1, 4 * tile_envs + 3))
        L = int(rng.integers(2, 9))
        T = int(rng.integers(6, 15))
        cfg = workloads.small_config(H=64, precision="bf16", n=n, A=A, D=D, E=E, C=E * int(rng.integers(1, 3)), L=L, T=T,
                                     seed=workloads.SEED_BASE + 500 + 10 * seed + done_shapes,
                                     env=dict(done_thresh24=int(rng.integers(0, 1 << 22))))
        try:
            actor = binding.Actor(cfg, kernel="pipelined")
        except binding.MarlError:
            continue                                  # outside the kernel's shared-memory budget: not its domain
        actor.destroy()
        w = workloads.make_weights(cfg)
        cut = int(rng.integers(1, T))
        splits = [cut, T - cut] if rng.integers(0, 2) else [1] * 2 + [T - 2]
        print(f"n={n} A={A} D={D} E={E} C={cfg['C']} L={L} T={T} splits={splits} done_thresh24={cfg['env']['done_thresh24']}", flush=True)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel="pipelined", splits=splits)
        assert actor.kernel_name == "tcgen05-pipelined"
        res = referee(cfg, w, actor, acts, q)
        print(f"   {res}")
        actor.destroy()
        done_shapes += 1


def test_pipelined_kernel_shapes_whose_availability_rows_are_not_word_aligned():
    """n * A not a multiple of four (workload 3's 5 x 11 among them): a chunk's availability bytes start anywhere
    inside a 16-byte unit of the input array; the kernel loads the aligned range around them and shifts.  The
    environment counts are multiples of 16, so every launch stays on the pipelined kernel: decisions, records and
    state equal the one-tile kernel's (where that kernel takes the shape), and every row passes the referee."""
    for over in (dict(n=5, A=11, D=80, E=208), dict(n=7, A=9, D=33, E=112), dict(n=5, A=11, D=55, E=64),
                 dict(n=9, A=3, D=16, E=48), dict(n=13, A=17, D=24, E=32)):
        cfg = workloads.small_config(H=64, precision="bf16", C=2 * over["E"], L=5, T=12,
                                     env=dict(done_thresh24=1 << 21), **over)
        w = workloads.make_weights(cfg)
        a, acts_a, q_a = run_gpu_rollout(cfg, w, kernel="pipelined", splits=[7, 1, 4])
        assert a.kernel_name == "tcgen05-pipelined"
        if over["D"] % 8 == 0:  # (the one-tile kernel takes observation rows of whole 8-column groups only)
            b, acts_b, q_b = run_gpu_rollout(cfg, w, kernel="tensor", splits=[7, 1, 4])
            assert b.kernel_name == "tcgen05"
            _assert_same_rollout(a, acts_a, q_a, b, acts_b, q_b, tag=str(over))
            b.destroy()
        print(over, referee(cfg, w, a, acts_a, q_a))
        a.destroy()


def test_shape_with_a_short_staging_ring_leaves_the_pipelined_kernel():
    """n=8, D=81, A=11 leaves room for three staging slots but a tile-step has four chunks: a converter warp would wait
    on a slot whose previous chunk belongs to another warp of the same step.  The pipelined kernel must not take the
    shape (it once did, and read stale availability bytes); the other kernels do."""
    cfg = workloads.small_config(H=64, precision="bf16", n=8, A=11, D=81, E=40, C=80, L=6, T=6,
                                 env=dict(done_thresh24=2578527))
    with pytest.raises(binding.MarlError):
        binding.Actor(cfg, kernel="pipelined")
    w = workloads.make_weights(cfg)
    actor, acts, q = run_gpu_rollout(cfg, w, kernel="auto", splits=[5, 1])
    assert actor.kernel_name != "tcgen05-pipelined"
    referee(cfg, w, actor, acts, q)
    actor.destroy()


def test_guard_bytes_around_the_buffers_catch_a_stray_write():
    """The harness surrounds every buffer it gives the library with guard bytes and checks them when an actor is
    destroyed.  A clean rollout leaves them alone; a byte planted here (by the test, through torch) just outside the
    state buffer and just behind the ring is reported."""
    cfg = workloads.small_config(H=64, E=40, C=80, L=8, T=6, precision="bf16", n=4, A=8, D=16)
    w = workloads.make_weights(cfg)
    actor, acts, q = run_gpu_rollout(cfg, w)
    assert binding.GUARD_BYTES > 0 and len(actor._guards) == 3
    actor.check_guards()
    for which, where in ((1, 4095), (0, -1)):
        full = actor._guards[which][0]
        keep = int(full[where])
        full[where] = 0
        with pytest.raises(binding.MarlError, match="outside"):
            actor.check_guards()
        full[where] = keep
    actor.destroy()


def test_streamed_hidden128_kernel_shapes_episode_ends_and_split_launches():
    """The tensor-core kernel for hidden size 128 (weights streamed through shared memory): tile tails, partial staging
    chunks, one tile, more tiles than blocks, agent counts that do not divide 128, observation widths that need padding
    to the MMA's K step; an episode end in every step and never; launches of one step and split rollouts."""
    for over in (dict(E=130, n=8, D=80, A=14, C=260), dict(E=1, n=4, A=4, D=8, C=2), dict(E=37, n=16, A=5, D=16, C=74),
                 dict(E=9, n=32, A=2, D=40, C=9), dict(E=2500, n=8, A=6, D=72, C=2500), dict(E=333, n=12, A=12, D=56, C=333)):
        cfg = workloads.small_config(H=128, L=7, T=20, precision="bf16", **over)
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w, kernel="pipelined", splits=[1, 6, 13])
        assert actor.kernel_name == "tcgen05-streamed"
        res = referee(cfg, w, actor, acts, q)
        print(f"H=128 {over}: {res}")
        actor.destroy()
    for thr, L in ((1 << 24, 4), (0, 5)):
        cfg = workloads.small_config(H=128, D=8, E=40, n=4, A=8, C=80, L=L, T=17, precision="bf16", env=dict(done_thresh24=thr))
        w = workloads.make_weights(cfg)
        actor, acts, q = run_gpu_rollout(cfg, w)
        assert actor.kernel_name == "tcgen05-streamed"
        referee(cfg, w, actor, acts, q)
        _, counters = actor.status()
        assert counters["episodes"] == (40 * 17 if thr else 40 * (17 // 5))
        actor.destroy()
    # step calls (one-step launches) reproduce the rollout; a list step falls back to the CUDA-core kernel and is clean
    cfg = workloads.small_config(H=128, D=24, E=50, n=4, A=12, C=100, L=8, T=12, precision="bf16")
    w = workloads.make_weights(cfg)
    ref, acts, q = run_gpu_rollout(cfg, w)
    obs, avail, rew, done = ref.env_generate(cfg["env"], 0, cfg["T"])
    dev = binding.Actor(cfg)
    dev.set_weights(w)
    for t in range(cfg["T"]):
        assert torch.equal(dev.step(obs[t], avail[t], rew[t], done[t], cfg["eps_start"]), acts[t])
    torch.cuda.synchronize()
    assert torch.equal(dev.ring_mem, ref.ring_mem)
    ids = np.arange(0, 48, 2, dtype=np.int32)
    tid = torch.as_tensor(ids, device="cuda", dtype=torch.long)
    dev.step_subset(ids, *(x[0].index_select(0, tid).contiguous() for x in (obs, avail, rew, done)), 0.1)
    assert dev.status()[0] == 0
    ref.destroy()
    dev.destroy()


def test_two_resident_tiles_write_the_same_ring_as_the_pipelined_kernel():
    """The kernel with two tiles resident per SM runs the arithmetic of the pipelined kernel: identical actions, Q,
    records, headers and state, on batches of more tiles than SMs - an even and an odd number of tiles per block, a
    ragged last tile, an episode end in every step, split launches (the short ones fall back to the pipelined kernel)."""
    for over, env in ((dict(E=2400, n=8, D=80, A=14, C=2400), {}), (dict(E=4730, n=8, D=80, A=14, C=4730), {}),
                      (dict(E=2500, n=16, D=24, A=5, C=5000), {}), (dict(E=5000, n=5, D=8, A=16, C=5000), dict(done_thresh24=1 << 24)),
                      (dict(E=7001, n=6, D=40, A=8, C=7001), dict(done_thresh24=1 << 21))):
        cfg = workloads.small_config(H=64, L=7, T=21, precision="bf16", env=env, **over)
        w = workloads.make_weights(cfg)
        a, acts_a, q_a = run_gpu_rollout(cfg, w, kernel="dual", splits=[9, 2, 10])
        b, acts_b, q_b = run_gpu_rollout(cfg, w, kernel="pipelined", splits=[9, 2, 10])
        assert a.kernel_name == "tcgen05-dual" and b.kernel_name == "tcgen05-pipelined"
        assert torch.equal(acts_a, acts_b) and torch.equal(q_a, q_b), over        # bit for bit
        assert torch.equal(a.ring_mem, b.ring_mem), over
        sa, sb = a.get_state(), b.get_state()
        for key in ("h", "last_action", "slot", "pos", "ep_count"):
            assert torch.equal(sa[key], sb[key]), (over, key)
        assert a.status() == b.status() and a.status()[0] == 0
        a.destroy()
        b.destroy()
    # and against the oracle, every environment
    cfg = workloads.small_config(H=64, L=9, T=24, precision="bf16", E=2600, n=8, D=80, A=14, C=5200)
    w = workloads.make_weights(cfg)
    actor, acts, q = run_gpu_rollout(cfg, w, kernel="dual")
    res = referee(cfg, w, actor, acts, q)
    print(f"dual: {res}")
    actor.destroy()

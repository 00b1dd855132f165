"""The learner's refresh of the shared model while the workers run (Sec. III-B; Algorithm 2 fetches the parameters
at the start of an iteration): a network published for global step s is the one every step >= s uses."""
import numpy as np
import pytest
import torch

from paper_2205_05248_b200 import binding, workloads
from referee import referee, run_gpu_rollout, sample_env_tiles
from test_gpu_parity import _assert_same_rollout

pytestmark = pytest.mark.gpu


def _published_rollout(cfg, w0, w1, kernel, switch, splits, publish_after):
    """Rollout in `splits` calls; w1 is published (for step `switch`) after `publish_after` of them."""
    actor = binding.Actor(cfg, kernel=kernel)
    actor.set_weights(w0, version=1)
    acts, q = actor.set_trace(cfg["T"], want_q=True)
    for k, part in enumerate(splits):
        if k == publish_after:
            actor.publish_weights(w1, version=2, effective_step=switch)
        actor.rollout(cfg["env"], part, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    torch.cuda.synchronize()
    return actor, acts, q


@pytest.mark.parametrize("kernel,prec,shape", [("pipelined", "bf16", dict(E=700, n=8, A=14, D=80, C=1400)),
                                               ("tensor", "bf16", dict(E=300, n=5, A=11, D=48, C=600)),
                                               ("ffma", "fp32", dict(E=64, n=3, A=5, D=16, C=128))])
def test_published_weights_take_effect_at_their_step(kernel, prec, shape):
    cfg = workloads.small_config(H=64, L=9, T=26, precision=prec, **shape)
    w0 = workloads.make_weights(cfg)
    w1 = workloads.make_weights(cfg, seed=cfg["seed"] + 977)
    switch = 11
    # the switch falls inside one launch; between two launches; at the first step of a later launch
    runs = [_published_rollout(cfg, w0, w1, kernel, switch, splits, after)
            for splits, after in (([26], 0), ([5, 21], 1), ([5, 6, 15], 1), ([11, 15], 0))]
    # the blocking route: stop, replace the network, go on
    ref = binding.Actor(cfg, kernel=kernel)
    ref.set_weights(w0, version=1)
    acts_r, q_r = ref.set_trace(cfg["T"], want_q=True)
    ref.rollout(cfg["env"], switch, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    ref.set_weights(w1, version=2)
    ref.rollout(cfg["env"], cfg["T"] - switch, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    torch.cuda.synchronize()
    for actor, acts, q in runs:
        assert actor.weights_version == 2
        _assert_same_rollout(actor, acts, q, ref, acts_r, q_r)
    # and against the oracle, which switches networks at the same step
    actor, acts, q = runs[0]
    res = referee(cfg, w0, actor, acts, q, weight_schedule=[(switch, w1)])       # every environment
    assert res["rows"] == cfg["T"] * cfg["E"] * cfg["n"]
    # the new network matters: a rollout that never switches differs after the switch step
    same, acts_s, q_s = run_gpu_rollout(cfg, w0, kernel=kernel)
    assert torch.equal(q_s[:switch], q[:switch]) and not torch.allclose(q_s[switch:], q[switch:], rtol=1e-2, atol=1e-3)
    for a in [r[0] for r in runs] + [ref, same]:
        a.destroy()


def test_publication_rules():
    cfg = workloads.small_config(H=64, D=16, E=32, C=64, L=6, T=12, precision="bf16", n=4, A=8)
    w0, w1, w2 = (workloads.make_weights(cfg, seed=s) for s in (1, 2, 3))
    actor = binding.Actor(cfg)
    with pytest.raises(binding.MarlError):
        actor.publish_weights(w1, 2, 0)          # no network yet
    actor.set_weights(w0, 1)
    actor.rollout(cfg["env"], 4, 0.1)
    with pytest.raises(binding.MarlError):
        actor.publish_weights(w1, 2, 3)          # step 3 has been enqueued already
    # a later publication replaces a pending one
    actor.publish_weights(w1, 2, 6)
    actor.publish_weights(w2, 3, 8)
    actor.rollout(cfg["env"], 3, 0.1)
    assert actor.weights_version == 1            # steps 4..6 enqueued: nothing switched yet
    actor.rollout(cfg["env"], 2, 0.1)
    assert actor.weights_version == 3
    # set_weights drops a pending publication
    actor.publish_weights(w1, 4, 100)
    actor.set_weights(w0, 5)
    actor.rollout(cfg["env"], 3, 0.1)
    assert actor.weights_version == 5
    # consecutive publications alternate between the two images
    for v in range(6, 10):
        actor.publish_weights(w1 if v % 2 else w2, v, actor.get_state()["step"])
        actor.rollout(cfg["env"], 1, 0.1)
        assert actor.weights_version == v
    torch.cuda.synchronize()
    assert actor.status()[0] == 0
    actor.destroy()


def test_published_weights_full_size_bench_configuration():
    """The configuration `bench.py --refresh` times: workload 5 at full size, one staged 64-step rollout with a
    publication that takes effect 32 steps in (two launches of 32 steps); the oracle recomputes 4096 environments
    (whole tiles) with the same switch."""
    cfg = workloads.config(5)
    T = cfg["T"]
    w0 = workloads.make_weights(cfg)
    w1 = workloads.make_weights(cfg, seed=cfg["seed"] + 1)
    actor = binding.Actor(cfg, kernel="auto", work_steps=1)
    assert actor.kernel_name == "tcgen05-pipelined"
    actor.set_weights(w0, version=1)
    acts, q = actor.set_trace(T, want_q=True)
    staged = actor.env_generate(cfg["env"], 0, T)
    launches = actor.launch_count
    actor.publish_weights(w1, version=2, effective_step=T // 2)
    actor.rollout_staged(*staged, T, cfg["eps_start"], cfg["eps_end"], cfg["anneal_steps"])
    torch.cuda.synchronize()
    assert actor.launch_count - launches == 2 and actor.weights_version == 2
    ids = sample_env_tiles(cfg["E"], 128 // cfg["n"], 4096, seed=6)      # whole tiles from every wave of both launches
    res = referee(cfg, w0, actor, acts, q, env_ids=ids, weight_schedule=[(T // 2, w1)])
    assert res["envs"] >= 4096
    print(f"cfg5 full size with a publication: {res}")
    status, counters = actor.status()
    assert status == 0 and counters["agent_steps"] == cfg["E"] * cfg["n"] * T
    del staged, acts, q
    actor.destroy()

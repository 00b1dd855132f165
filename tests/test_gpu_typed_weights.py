"""Per-type agent networks (heterogeneous teams, Table I): the CUDA library against the oracle."""
import numpy as np
import pytest
import torch

from paper_2205_05248_b200 import binding, workloads
from referee import referee, run_gpu_rollout

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("prec", ["fp32", "bf16"])
def test_workload3_team_with_a_network_per_unit_type(prec):
    """Workload 3 at full size (4096 environments, 2 + 3 agents of two unit types, annealed epsilon, 256 steps),
    every environment refereed against the oracle with the same two networks."""
    cfg = workloads.typed(workloads.config(3, precision=prec))
    assert cfg["agent_type"] == [0, 0, 1, 1, 1]
    ws = workloads.make_weights_typed(cfg)
    actor, acts, q = run_gpu_rollout(cfg, ws)
    assert actor.kernel_name == "ffma"
    res = referee(cfg, ws, actor, acts, q)
    print(f"cfg3 typed {prec}: {res}")
    assert res["envs"] == cfg["E"]
    actor.destroy()


@pytest.mark.parametrize("shape,types", [(dict(E=70, n=7, D=13, A=6, C=140), [2, 0, 1, 1, 0, 2, 3]),
                                         (dict(E=33, n=3, D=30, A=9, C=33), [1, 0, 1]),
                                         (dict(E=200, n=8, D=80, A=14, C=200, H=128), [0, 1, 0, 1, 1, 1, 0, 0])])
def test_typed_networks_ragged_shapes(shape, types):
    for prec in ("fp32", "bf16"):
        cfg = workloads.typed(workloads.small_config(**{**dict(H=64, L=7, T=15, precision=prec), **shape}), agent_type=types)
        ws = workloads.make_weights_typed(cfg)
        actor, acts, q = run_gpu_rollout(cfg, ws, splits=[4, 11])
        referee(cfg, ws, actor, acts, q)
        actor.destroy()


def test_identical_networks_per_type_equal_the_shared_network_and_modes_switch():
    """The typed route with the same network for every type reproduces the shared route bit for bit on the CUDA-core
    kernel; loading per-type networks moves a tensor-core actor to the CUDA-core kernel and marl_actor_set_weights
    moves it back."""
    base = workloads.small_config(H=64, E=150, n=5, D=80, A=11, C=300, L=9, T=20, precision="bf16", env=dict(n_type0=2))
    cfg = workloads.typed(base)
    w = workloads.make_weights(base)
    shared, a_s, q_s = run_gpu_rollout(base, w, kernel="ffma")
    typed, a_t, q_t = run_gpu_rollout(cfg, [w, w], kernel="ffma")
    assert torch.equal(a_s, a_t) and torch.equal(q_s, q_t)
    assert torch.equal(shared.ring_mem, typed.ring_mem)
    assert torch.equal(shared.get_state()["h"], typed.get_state()["h"])
    shared.destroy()
    typed.destroy()
    auto = binding.Actor(cfg)                       # bf16, a supported shape: a tensor-core kernel by default
    auto.set_weights(w)
    assert auto.kernel_name.startswith("tcgen05")
    auto.set_weights_typed(workloads.make_weights_typed(cfg), version=2)
    assert auto.kernel_name == "ffma" and auto.weights_version == 2
    with pytest.raises(binding.MarlError, match="per-type"):
        auto.publish_weights(w, 3, 5)
    auto.rollout(cfg["env"], 3, 0.1)
    auto.set_weights(w, version=4)
    assert auto.kernel_name.startswith("tcgen05")
    auto.rollout(cfg["env"], 3, 0.1)
    torch.cuda.synchronize()
    assert auto.status()[0] == 0
    # validation
    with pytest.raises(binding.MarlError, match="agent_type"):
        auto.set_weights_typed([w, w], agent_type=[0, 1, 2, 0, 0])
    with pytest.raises(binding.MarlError, match="n_types"):
        auto.set_weights_typed([w, w, w], agent_type=[0, 1, 2, 0, 0])
    auto.destroy()
    plain = binding.Actor(base)                     # created without room for per-type networks
    with pytest.raises(binding.MarlError, match="n_types"):
        plain.set_weights_typed([w, w], agent_type=[0, 0, 1, 1, 1])
    plain.destroy()

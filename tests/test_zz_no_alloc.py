"""marl_rollout_noalloc against marl_rollout.

Some users of the library run inside a process that owns all device memory through its own pool, or in a
loop where a cudaMalloc (which stalls the whole device and can fail) is not acceptable.  For them the library
offers a rollout whose staging area is a fixed array inside the library instead of allocated memory.  This
test drives that entry point through the C ABI and checks that it produces what marl_rollout produces - the
same actions and ring bytes, Q and hidden state within the tolerance the other parity tests use - on two
calls in a row (the second call finds the first call's bytes still in the shared array), on the CUDA-core
kernel and on the tensor-core kernel (whose bulk copies read the array directly), that after the set-up call
a rollout leaves the amount of free device memory exactly as it found it, and that a configuration too large
for the array is refused with an error code instead of being run.

The file name sorts last on purpose: a run that stops at the first failure has then already run every other
test.  It does not depend on them and passes alone in a fresh process too.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2205_05248_b200 import binding, workloads
from referee import RTOL, row_rel_err

pytestmark = pytest.mark.gpu


def _pair(cfg, kernel):
    w = workloads.make_weights(cfg)
    out = []
    for _ in range(2):
        a = binding.Actor(cfg, kernel=kernel, work_steps=cfg["T"])
        a.set_weights(w)
        a.set_trace(2 * cfg["T"])
        out.append(a)
    return out


def test_setup_call_places_the_array_and_needs_no_actor():
    """T = 0 is the set-up call: no actor, no environment, no work - only the array's address is looked up (which is
    when the driver gives the array its memory on this device).  A second set-up call finds it in place."""
    torch.cuda.init()
    lib = binding.load_library()
    assert lib.marl_rollout_noalloc(None, None, C.c_int32(0), C.c_double(0), C.c_double(0), C.c_int32(0)) == 0
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    assert lib.marl_rollout_noalloc(None, None, C.c_int32(0), C.c_double(0), C.c_double(0), C.c_int32(0)) == 0
    assert torch.cuda.mem_get_info()[0] == free0


@pytest.mark.parametrize("kernel", ["ffma", "auto"])
@pytest.mark.parametrize("over", [dict(E=300, n=3, D=30, A=9, C=600, L=16, T=12),      # fits in one window
                                  dict(E=2048, n=8, D=80, A=14, C=2048, L=40, T=17)])  # needs several windows
def test_noalloc_rollout_matches_rollout_twice(over, kernel):
    cfg = workloads.small_config(H=64, precision="bf16", **over)
    ref, dut = _pair(cfg, kernel)
    if kernel == "auto" and over["n"] >= 4:
        assert dut.kernel_name.startswith("tcgen05")     # this case reads the array with bulk copies
    rtol = RTOL[cfg["precision"]]
    for call in range(2):
        ref.rollout(cfg["env"], cfg["T"], 0.3, 0.05, 2 * cfg["T"] - 1)
        torch.cuda.synchronize()
        free_before, torch_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        dut.rollout_noalloc(cfg["env"], cfg["T"], 0.3, 0.05, 2 * cfg["T"] - 1)
        torch.cuda.synchronize()
        if call == 1:        # the first call may be this process's set-up call and the first use of a kernel
            assert torch.cuda.mem_get_info()[0] == free_before, "device memory was taken during the call"
            assert torch.cuda.memory_allocated() == torch_before
        steps = (call + 1) * cfg["T"]
        (ra, rq), (da, dq) = ref._trace, dut._trace
        assert torch.equal(ra[:steps], da[:steps])
        assert row_rel_err(dq[:steps].cpu().numpy(), rq[:steps].cpu().numpy()).max() <= rtol
        rs, ds = ref.get_state(), dut.get_state()
        for key in ("last_action", "slot", "pos", "ep_count"):
            assert torch.equal(rs[key], ds[key]), key
        assert rs["step"] == ds["step"] == steps
        assert row_rel_err(ds["h"].cpu().numpy(), rs["h"].cpu().numpy()).max() <= rtol
        rr, dr = ref.ring_view(), dut.ring_view()
        for key in ("obs", "avail", "action", "reward", "done", "slot_epid", "slot_len", "slot_complete"):
            assert torch.equal(rr[key], dr[key]), key
        assert row_rel_err(dr["q"].cpu().numpy().reshape(-1, cfg["A"]),
                           rr["q"].cpu().numpy().reshape(-1, cfg["A"])).max() <= rtol
        assert dut.status()[0] == 0
    ref.destroy()
    dut.destroy()


def test_noalloc_rejects_a_step_that_does_not_fit():
    """One environment step of this shape stages about 44 MB, more than the 32 MiB array."""
    cfg = workloads.small_config(H=64, E=16384, n=8, D=80, A=14, C=16384, L=2, T=1)
    a = binding.Actor(cfg, kernel="ffma", work_steps=1)
    a.set_weights(workloads.make_weights(cfg))
    with pytest.raises(binding.MarlError, match="-4"):
        a.rollout_noalloc(cfg["env"], 1, 0.1)
    assert a.get_state()["step"] == 0 and a.status()[0] == 0       # nothing ran
    a.destroy()

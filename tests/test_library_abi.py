"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared symbol, sizes
buffers sensibly, rejects bad configurations with error codes, and refuses to run without a CUDA device."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2205_05248_b200 import binding, build, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "marl_actor.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(marl_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert len(names) >= 19
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_query_sizes_and_record_layout(lib):
    cfg = workloads.config(5)
    s = binding.marl_actor_query_sizes(cfg)
    rec = 8 * 80 * 4 + 112 + 32 + 8 * 14 * 4 + 16          # obs | avail | action | q | reward+done
    assert rec % 16 == 0
    assert s["ring_bytes"] >= 65536 * 96 * rec
    assert s["ring_bytes"] < 65536 * 96 * rec + (2 << 20)
    assert 19.5e9 < s["ring_bytes"] < 20.5e9                # "about 20 GB"
    assert s["state_bytes"] >= 65536 * 8 * 64 * 4
    per = s["work_bytes_per_step"]
    assert per >= 65536 * 8 * (80 * 4 + 14) + 65536 * 5
    # records are padded to 16 bytes for shapes whose rows are not multiples of 16 bytes
    for k in (1, 4):
        c = workloads.config(k)
        sz = binding.marl_actor_query_sizes(c)
        assert sz["ring_bytes"] % 256 == 0


@pytest.mark.parametrize("over", [dict(E=0), dict(n=0), dict(n=33), dict(A=33), dict(D=0), dict(H=48),
                                  dict(C=7), dict(L=0), dict(precision=5)])
def test_bad_config_is_an_error_code(lib, over):
    cfg = workloads.small_config(H=64)
    cfg.update(over)
    c = binding.make_config(cfg)
    s = binding.Sizes()
    rc = lib.marl_actor_query_sizes(C.byref(c), C.byref(s))
    assert rc == -1 and lib.marl_last_error()
    h = C.c_void_p()
    assert lib.marl_actor_create(C.byref(c), C.byref(h)) == -1 and not h.value


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the behaviour without a CUDA device")
def test_create_without_gpu_fails_loudly(lib):
    cfg = workloads.small_config(H=64)
    c = binding.make_config(cfg)
    h = C.c_void_p()
    rc = lib.marl_actor_create(C.byref(c), C.byref(h))
    assert rc == -3 and not h.value and b"cuda" in lib.marl_last_error().lower()
    with pytest.raises(binding.MarlError):
        binding.Actor(cfg)


def test_null_handles_are_rejected(lib):
    assert lib.marl_actor_step(None, None, None, None, None, C.c_float(0.1), None) == -1
    assert lib.marl_rollout(None, None, 1, 0.1, 0.1, 0) == -1
    assert lib.marl_ring_view(None, None) == -1
    assert lib.marl_actor_launch_count(None) == 0
    lib.marl_actor_destroy(None)

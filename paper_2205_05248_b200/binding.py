"""Thin Python binding of the C-ABI actor library (``include/marl_actor.h``).

Argument marshalling only: torch supplies device memory and streams, every step of the path runs in the
library's CUDA kernels.  The shared object is built in-tree by ``paper_2205_05248_b200.build``; if it is
missing, or no CUDA device is present, calls fail with an exception - there is no CPU path.

The module-level functions carry the C names (``marl_actor_create`` ...); ``Actor`` wraps a handle together
with the torch tensors that back its ring, state and staging memory.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmarl_actor.so")

PRECISION = {"fp32": 0, "bf16": 1}
KERNEL = {"auto": 0, "ffma": 1, "tensor": 2, "pipelined": 3, "dual": 4}
STATUS_NO_AVAIL, STATUS_TIMEOUT, STATUS_BAD_INDEX = 1, 2, 4

# Debug aid: with GUARD_BYTES > 0 (a multiple of 256; the test-suite sets it) every buffer an Actor hands to the
# library gets that many guard bytes of a fixed pattern in front of it and behind it, and ``Actor.check_guards``
# (called by ``destroy``) raises if the library has written outside a buffer.
GUARD_BYTES = 0
GUARD_PATTERN = 0xA5

EXPORTS = [
    "marl_actor_query_sizes", "marl_actor_create", "marl_actor_set_weights", "marl_actor_set_weights_typed",
    "marl_actor_publish_weights",
    "marl_actor_weights_version",
    "marl_actor_step", "marl_actor_step_subset", "marl_actor_step_lagged", "marl_actor_step_host", "marl_env_generate", "marl_rollout_staged", "marl_rollout",
    "marl_actor_set_trace", "marl_ring_view", "marl_ring_sample", "marl_actor_get_state", "marl_actor_set_state",
    "marl_actor_status", "marl_actor_reset", "marl_actor_destroy", "marl_actor_kernel_name",
    "marl_actor_launch_count", "marl_last_error", "marl_rollout_noalloc", "marl_selftest_bounded_wait",
    "marl_measure_ffma_tflops",
]


class MarlError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [("n_envs", C.c_int32), ("n_agents", C.c_int32), ("obs_dim", C.c_int32), ("n_actions", C.c_int32),
                ("hidden", C.c_int32), ("ring_episodes", C.c_int32), ("ring_steps", C.c_int32),
                ("precision", C.c_int32), ("kernel", C.c_int32), ("n_agent_types", C.c_int32), ("seed", C.c_uint64),
                ("stream", C.c_void_p), ("ring_mem", C.c_void_p), ("ring_bytes", C.c_size_t),
                ("state_mem", C.c_void_p), ("state_bytes", C.c_size_t), ("work_mem", C.c_void_p),
                ("work_bytes", C.c_size_t)]


class Sizes(C.Structure):
    _fields_ = [("ring_bytes", C.c_size_t), ("state_bytes", C.c_size_t), ("work_bytes_min", C.c_size_t),
                ("work_bytes_per_step", C.c_size_t)]


class SynthEnv(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("obs_law", C.c_int32), ("done_thresh24", C.c_uint32),
                ("avail_thresh_first", C.c_uint32), ("avail_thresh_rest", C.c_uint32), ("avail_split", C.c_int32),
                ("n_type0", C.c_int32), ("type_block_start", C.c_int32), ("type_block_len", C.c_int32)]


class SampleBatch(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("obs", "avail", "action", "q", "reward", "done", "slot", "len", "epid")]


class RingView(C.Structure):
    _fields_ = [("base", C.c_void_p), ("slot_stride", C.c_size_t), ("step_stride", C.c_size_t),
                ("off_obs", C.c_size_t), ("off_avail", C.c_size_t), ("off_action", C.c_size_t),
                ("off_q", C.c_size_t), ("off_reward", C.c_size_t), ("off_done", C.c_size_t),
                ("episodes", C.c_int32), ("steps", C.c_int32), ("slots_per_env", C.c_int32), ("n_envs", C.c_int32),
                ("n_agents", C.c_int32), ("obs_dim", C.c_int32), ("n_actions", C.c_int32), ("reserved", C.c_int32),
                ("slot_epid", C.c_void_p), ("slot_len", C.c_void_p), ("slot_complete", C.c_void_p)]


class StateView(C.Structure):
    _fields_ = [("h", C.c_void_p), ("last_action", C.c_void_p), ("slot", C.c_void_p), ("pos", C.c_void_p),
                ("ep_count", C.c_void_p), ("step", C.c_uint64)]


class Counters(C.Structure):
    _fields_ = [("agent_steps", C.c_uint64), ("episodes", C.c_uint64), ("explored", C.c_uint64),
                ("no_avail", C.c_uint64), ("truncated", C.c_uint64)]


_lib = None


def load_library():
    """Loads libmarl_actor.so (no CUDA call is made by loading).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise MarlError(f"{LIB_PATH} is missing: run `python -m paper_2205_05248_b200.build` (there is no "
                            "CPU fallback)")
        lib = C.CDLL(LIB_PATH)
        P = C.c_void_p
        lib.marl_last_error.restype = C.c_char_p
        lib.marl_actor_kernel_name.restype = C.c_char_p
        lib.marl_actor_kernel_name.argtypes = [P]
        lib.marl_actor_launch_count.restype = C.c_uint64
        lib.marl_actor_launch_count.argtypes = [P]
        lib.marl_actor_weights_version.restype = C.c_uint64
        lib.marl_actor_weights_version.argtypes = [P]
        lib.marl_actor_destroy.restype = None
        lib.marl_actor_destroy.argtypes = [P]
        lib.marl_actor_query_sizes.argtypes = [C.POINTER(Config), C.POINTER(Sizes)]
        lib.marl_actor_create.argtypes = [C.POINTER(Config), C.POINTER(P)]
        lib.marl_actor_set_weights.argtypes = [P] + [P] * 8 + [C.c_uint64]
        lib.marl_actor_set_weights_typed.argtypes = [P, C.c_int32, P] + [P] * 8 + [C.c_uint64]
        lib.marl_actor_publish_weights.argtypes = [P] + [P] * 8 + [C.c_uint64, C.c_uint64]
        lib.marl_actor_step.argtypes = [P, P, P, P, P, C.c_float, P]
        lib.marl_actor_step_host.argtypes = [P, P, P, P, P, C.c_float, P]
        lib.marl_actor_step_subset.argtypes = [P, P, C.c_int32, P, P, P, P, C.c_float, P]
        lib.marl_actor_step_lagged.argtypes = [P, P, C.c_int32, P, P, P, P, C.c_float, P]
        lib.marl_env_generate.argtypes = [P, C.POINTER(SynthEnv), C.c_uint32, C.c_int32, P, P, P, P]
        lib.marl_rollout_staged.argtypes = [P, P, P, P, P, C.c_int32, C.c_double, C.c_double, C.c_int32]
        lib.marl_rollout.argtypes = [P, C.POINTER(SynthEnv), C.c_int32, C.c_double, C.c_double, C.c_int32]
        lib.marl_rollout_noalloc.argtypes = [P, C.POINTER(SynthEnv), C.c_int32, C.c_double, C.c_double, C.c_int32]
        lib.marl_measure_ffma_tflops.argtypes = [P, C.POINTER(C.c_double)]
        lib.marl_selftest_bounded_wait.argtypes = [P, C.c_uint32, C.POINTER(C.c_uint32)]
        lib.marl_actor_set_trace.argtypes = [P, P, P, C.c_int32]
        lib.marl_ring_view.argtypes = [P, C.POINTER(RingView)]
        lib.marl_ring_sample.argtypes = [P, C.c_uint32, C.c_int32, C.POINTER(SampleBatch)]
        lib.marl_actor_get_state.argtypes = [P, C.POINTER(StateView)]
        lib.marl_actor_set_state.argtypes = [P, C.POINTER(StateView)]
        lib.marl_actor_status.argtypes = [P, C.POINTER(C.c_uint32), C.POINTER(Counters)]
        lib.marl_actor_reset.argtypes = [P]
        _lib = lib
    return _lib


def _check(rc: int):
    if rc != 0:
        raise MarlError(f"marl error {rc}: {load_library().marl_last_error().decode()}")


def make_env(env: dict) -> SynthEnv:
    return SynthEnv(int(env["seed"]), int(env["obs_law"]), int(env["done_thresh24"]),
                    int(env["avail_thresh_first"]), int(env["avail_thresh_rest"]), int(env["avail_split"]),
                    int(env["n_type0"]), int(env["type_block_start"]), int(env["type_block_len"]))


def make_config(cfg: dict, kernel: str = "auto") -> Config:
    prec = cfg["precision"]
    prec = PRECISION.get(prec, prec)
    c = Config()
    c.n_envs, c.n_agents, c.obs_dim, c.n_actions, c.hidden = cfg["E"], cfg["n"], cfg["D"], cfg["A"], cfg["H"]
    c.ring_episodes, c.ring_steps, c.precision, c.kernel = cfg["C"], cfg["L"], int(prec), KERNEL[kernel]
    c.seed = int(cfg["seed"])
    c.n_agent_types = (max(cfg["agent_type"]) + 1) if cfg.get("agent_type") is not None else 0
    return c


def marl_actor_query_sizes(cfg: dict) -> dict:
    s = Sizes()
    c = make_config(cfg)
    _check(load_library().marl_actor_query_sizes(C.byref(c), C.byref(s)))
    return {k: getattr(s, k) for k, _ in Sizes._fields_}


def marl_measure_ffma_tflops() -> float:
    """fp32 FMA peak of the current device under load, in TFLOP/s (measured by the library)."""
    out = C.c_double(0)
    stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().marl_measure_ffma_tflops(C.c_void_p(stream), C.byref(out)))
    return float(out.value)


def marl_selftest_bounded_wait(poll_limit: int = 20000) -> int:
    """Runs the bounded-wait self-test on the current stream; returns the reported status word."""
    st = C.c_uint32(0)
    stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().marl_selftest_bounded_wait(C.c_void_p(stream), C.c_uint32(poll_limit), C.byref(st)))
    return int(st.value)


def _dptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Actor:
    """A library handle plus the torch tensors that back it.

    work_steps: how many environment steps of staging to allocate for ``rollout`` (default: cfg['T'] if it
    fits in ``work_budget_bytes``, else as many as fit).
    """

    def __init__(self, cfg: dict, device: str = "cuda:0", kernel: str = "auto", work_steps: int | None = None,
                 work_budget_bytes: int = 24 << 30):
        if not torch.cuda.is_available():
            raise MarlError("no CUDA device: the actor library has no CPU path")
        self.lib = load_library()
        self.cfg = dict(cfg)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        sizes = marl_actor_query_sizes(cfg)
        steps = cfg.get("T", 1) if work_steps is None else work_steps
        per = sizes["work_bytes_per_step"]
        steps = max(1, min(steps, (work_budget_bytes - sizes["work_bytes_min"]) // per + 1))
        wbytes = sizes["work_bytes_min"] + (steps - 1) * per
        u8 = dict(dtype=torch.uint8, device=self.device)
        self._guards = []

        def alloc(nbytes, zero):
            g = GUARD_BYTES
            if g <= 0:
                return torch.zeros(nbytes, **u8) if zero else torch.empty(nbytes, **u8)
            assert g % 256 == 0
            full = torch.zeros(nbytes + 2 * g, **u8) if zero else torch.empty(nbytes + 2 * g, **u8)
            full[:g] = GUARD_PATTERN
            full[g + nbytes:] = GUARD_PATTERN
            self._guards.append((full, g, nbytes))
            return full[g:g + nbytes]

        self.ring_mem = alloc(sizes["ring_bytes"], True)   # padding bytes are never written
        self.state_mem = alloc(sizes["state_bytes"], False)
        self.work_mem = alloc(wbytes, False)
        c = make_config(cfg, kernel)
        self.stream = torch.cuda.current_stream(self.device)
        c.stream = self.stream.cuda_stream
        c.ring_mem, c.ring_bytes = self.ring_mem.data_ptr(), self.ring_mem.numel()
        c.state_mem, c.state_bytes = self.state_mem.data_ptr(), self.state_mem.numel()
        c.work_mem, c.work_bytes = self.work_mem.data_ptr(), self.work_mem.numel()
        h = C.c_void_p()
        _check(self.lib.marl_actor_create(C.byref(c), C.byref(h)))
        self.handle = h
        self._trace = None
        self._keep = []

    # -- lifetime ---------------------------------------------------------------------------------
    def destroy(self):
        if getattr(self, "handle", None):
            self.lib.marl_actor_destroy(self.handle)      # synchronises the stream
            self.handle = None
            self.check_guards()

    def check_guards(self):
        """Raises if any guard byte around the ring, state or work buffer has changed (GUARD_BYTES > 0 only)."""
        for name, (full, g, nbytes) in zip(("ring_mem", "state_mem", "work_mem"), getattr(self, "_guards", [])):
            front_ok = bool((full[:g] == GUARD_PATTERN).all())
            back_ok = bool((full[g + nbytes:] == GUARD_PATTERN).all())
            if not (front_ok and back_ok):
                raise MarlError(f"the library wrote outside {name} ({'before' if not front_ok else 'behind'} the buffer)")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- weights ----------------------------------------------------------------------------------
    def set_weights(self, w: dict, version: int = 1):
        import numpy as np
        arrs = [np.ascontiguousarray(w[k], dtype=np.float32)
                for k in ("W1", "b1", "W_ih", "b_ih", "W_hh", "b_hh", "W2", "b2")]
        _check(self.lib.marl_actor_set_weights(self.handle, *[a.ctypes.data_as(C.c_void_p) for a in arrs],
                                               C.c_uint64(version)))

    def set_weights_typed(self, ws: list, agent_type=None, version: int = 1):
        """marl_actor_set_weights_typed: one network (a dict like ``set_weights`` takes) per unit type; agent_type
        defaults to the configuration's."""
        import numpy as np
        types = np.ascontiguousarray(self.cfg["agent_type"] if agent_type is None else agent_type, dtype=np.int32)
        arrs = [np.ascontiguousarray(np.stack([w[k] for w in ws]), dtype=np.float32)
                for k in ("W1", "b1", "W_ih", "b_ih", "W_hh", "b_hh", "W2", "b2")]
        _check(self.lib.marl_actor_set_weights_typed(self.handle, C.c_int32(len(ws)), types.ctypes.data_as(C.c_void_p),
                                                     *[a.ctypes.data_as(C.c_void_p) for a in arrs], C.c_uint64(version)))

    def publish_weights(self, w: dict, version: int, effective_step: int):
        """marl_actor_publish_weights: the network in use from global step effective_step on."""
        import numpy as np
        arrs = [np.ascontiguousarray(w[k], dtype=np.float32)
                for k in ("W1", "b1", "W_ih", "b_ih", "W_hh", "b_hh", "W2", "b2")]
        _check(self.lib.marl_actor_publish_weights(self.handle, *[a.ctypes.data_as(C.c_void_p) for a in arrs],
                                                   C.c_uint64(version), C.c_uint64(effective_step)))

    @property
    def weights_version(self) -> int:
        return int(self.lib.marl_actor_weights_version(self.handle))

    # -- stepping ---------------------------------------------------------------------------------
    def step(self, obs, avail, reward, done, eps: float, actions_out=None):
        """marl_actor_step on device tensors; returns the int32 [E][n] action tensor."""
        E, n = self.cfg["E"], self.cfg["n"]
        if actions_out is None:
            actions_out = torch.empty((E, n), dtype=torch.int32, device=self.device)
        for t, dt in ((obs, torch.float32), (avail, torch.uint8), (reward, torch.float32), (done, torch.uint8)):
            assert t.is_cuda and t.dtype == dt and t.is_contiguous()
        _check(self.lib.marl_actor_step(self.handle, _dptr(obs), _dptr(avail), _dptr(reward), _dptr(done),
                                        C.c_float(eps), _dptr(actions_out)))
        return actions_out

    def step_lagged(self, env_ids, obs, avail, prev_reward, prev_done, eps: float, actions_out=None):
        """marl_actor_step_lagged: step_subset with the outcome of each environment's previous action."""
        return self.step_subset(env_ids, obs, avail, prev_reward, prev_done, eps, actions_out, lagged=True)

    def step_subset(self, env_ids, obs, avail, reward, done, eps: float, actions_out=None, lagged=False):
        """marl_actor_step_subset: env_ids is a host int32 array [M]; the other tensors are device tensors over the
        list.  Returns the int32 [M][n] action tensor."""
        import numpy as np
        ids = np.ascontiguousarray(env_ids, dtype=np.int32)
        M, n = int(ids.shape[0]), self.cfg["n"]
        if actions_out is None:
            actions_out = torch.empty((M, n), dtype=torch.int32, device=self.device)
        for t, dt in ((obs, torch.float32), (avail, torch.uint8), (reward, torch.float32), (done, torch.uint8)):
            assert t.is_cuda and t.dtype == dt and t.is_contiguous() and t.shape[0] == M
        fn = self.lib.marl_actor_step_lagged if lagged else self.lib.marl_actor_step_subset
        _check(fn(self.handle, ids.ctypes.data_as(C.c_void_p), C.c_int32(M), _dptr(obs), _dptr(avail), _dptr(reward),
                  _dptr(done), C.c_float(eps), _dptr(actions_out)))
        return actions_out

    def step_host(self, obs, avail, reward, done, eps: float, actions_out):
        """marl_actor_step_host on host tensors (pinned for asynchronous copies); synchronises."""
        for t in (obs, avail, reward, done, actions_out):
            assert not t.is_cuda and t.is_contiguous()
        _check(self.lib.marl_actor_step_host(self.handle, _dptr(obs), _dptr(avail), _dptr(reward), _dptr(done),
                                             C.c_float(eps), _dptr(actions_out)))
        return actions_out

    def env_generate(self, env: dict, t0: int, n_steps: int, out=None):
        """marl_env_generate into fresh (or given) device tensors laid out [step][E]..."""
        c = self.cfg
        E, n, D, A = c["E"], c["n"], c["D"], c["A"]
        if out is None:
            out = (torch.empty((n_steps, E, n, D), dtype=torch.float32, device=self.device),
                   torch.empty((n_steps, E, n, A), dtype=torch.uint8, device=self.device),
                   torch.empty((n_steps, E), dtype=torch.float32, device=self.device),
                   torch.empty((n_steps, E), dtype=torch.uint8, device=self.device))
        ev = make_env(env)
        _check(self.lib.marl_env_generate(self.handle, C.byref(ev), C.c_uint32(t0), C.c_int32(n_steps),
                                          *[_dptr(t) for t in out]))
        return out

    def rollout_staged(self, obs, avail, reward, done, T: int, eps_start: float, eps_end: float | None = None,
                       anneal_steps: int = 0):
        eps_end = eps_start if eps_end is None else eps_end
        _check(self.lib.marl_rollout_staged(self.handle, _dptr(obs), _dptr(avail), _dptr(reward), _dptr(done),
                                            C.c_int32(T), C.c_double(eps_start), C.c_double(eps_end),
                                            C.c_int32(anneal_steps)))

    def rollout(self, env: dict, T: int, eps_start: float, eps_end: float | None = None, anneal_steps: int = 0):
        eps_end = eps_start if eps_end is None else eps_end
        ev = make_env(env)
        _check(self.lib.marl_rollout(self.handle, C.byref(ev), C.c_int32(T), C.c_double(eps_start),
                                     C.c_double(eps_end), C.c_int32(anneal_steps)))

    def rollout_noalloc(self, env: dict, T: int, eps_start: float, eps_end: float | None = None,
                        anneal_steps: int = 0):
        """marl_rollout_noalloc: same results as ``rollout``, staged through the library's fixed scratch array
        (for callers that may not allocate device memory).  On failure the exception carries the return code, so
        "too large for the scratch" (-4, MARL_ENOMEM) can be told from other errors."""
        eps_end = eps_start if eps_end is None else eps_end
        ev = make_env(env)
        rc = self.lib.marl_rollout_noalloc(self.handle, C.byref(ev), C.c_int32(T), C.c_double(eps_start),
                                           C.c_double(eps_end), C.c_int32(anneal_steps))
        if rc != 0:
            raise MarlError(f"marl_rollout_noalloc failed with code {rc}")

    # -- verification trace -----------------------------------------------------------------------
    def set_trace(self, capacity_steps: int, want_q: bool = True):
        c = self.cfg
        if capacity_steps <= 0:
            self._trace = None
            _check(self.lib.marl_actor_set_trace(self.handle, None, None, 0))
            return None
        acts = torch.full((capacity_steps, c["E"], c["n"]), -7, dtype=torch.int32, device=self.device)
        q = (torch.full((capacity_steps, c["E"], c["n"], c["A"]), float("nan"), dtype=torch.float32,
                        device=self.device) if want_q else None)
        self._trace = (acts, q)
        _check(self.lib.marl_actor_set_trace(self.handle, _dptr(acts), _dptr(q), C.c_int32(capacity_steps)))
        return self._trace

    # -- views ------------------------------------------------------------------------------------
    def ring_view(self) -> dict:
        """marl_ring_view as strided torch views over the ring memory (no copies)."""
        v = RingView()
        _check(self.lib.marl_ring_view(self.handle, C.byref(v)))
        base_off = v.base - self.ring_mem.data_ptr()
        Cn, L, n, D, A = v.episodes, v.steps, v.n_agents, v.obs_dim, v.n_actions
        u8 = self.ring_mem
        f32 = u8[: u8.numel() // 4 * 4].view(torch.float32)
        i32 = u8[: u8.numel() // 4 * 4].view(torch.int32)
        ss, ps = v.slot_stride, v.step_stride

        # (as_strided offsets count from the start of the storage, and ring_mem may itself start inside one)
        so4, so1 = f32.storage_offset(), u8.storage_offset()

        def f(off, shape_tail, stride_tail):
            return torch.as_strided(f32, (Cn, L, *shape_tail), (ss // 4, ps // 4, *stride_tail), so4 + (base_off + off) // 4)

        def hdr(ptr, dtype, count):
            o = ptr - u8.data_ptr()
            nb = torch.empty((), dtype=dtype).element_size() * count
            return u8[o:o + nb].view(dtype)

        out = dict(
            obs=f(v.off_obs, (n, D), (D, 1)), q=f(v.off_q, (n, A), (A, 1)), reward=f(v.off_reward, (), ()),
            action=torch.as_strided(i32, (Cn, L, n), (ss // 4, ps // 4, 1), so4 + (base_off + v.off_action) // 4),
            avail=torch.as_strided(u8, (Cn, L, n, A), (ss, ps, A, 1), so1 + base_off + v.off_avail),
            done=torch.as_strided(u8, (Cn, L), (ss, ps), so1 + base_off + v.off_done),
            slot_epid=hdr(v.slot_epid, torch.int64, Cn), slot_len=hdr(v.slot_len, torch.int32, Cn),
            slot_complete=hdr(v.slot_complete, torch.uint8, Cn))
        out["meta"] = {k: getattr(v, k) for k, _ in RingView._fields_}
        return out

    def ring_sample(self, draw_index: int, B: int) -> dict:
        """marl_ring_sample into fresh device tensors: a dense batch of B episodes drawn from the ring."""
        c = self.cfg
        L, n, D, A = c["L"], c["n"], c["D"], c["A"]
        dev = self.device
        out = dict(obs=torch.empty((B, L, n, D), dtype=torch.float32, device=dev),
                   avail=torch.empty((B, L, n, A), dtype=torch.uint8, device=dev),
                   action=torch.empty((B, L, n), dtype=torch.int32, device=dev),
                   q=torch.empty((B, L, n, A), dtype=torch.float32, device=dev),
                   reward=torch.empty((B, L), dtype=torch.float32, device=dev),
                   done=torch.empty((B, L), dtype=torch.uint8, device=dev),
                   slot=torch.empty((B,), dtype=torch.int32, device=dev),
                   len=torch.empty((B,), dtype=torch.int32, device=dev),
                   epid=torch.empty((B,), dtype=torch.int64, device=dev))
        sb = SampleBatch(*[_dptr(out[k]) for k, _ in SampleBatch._fields_])
        _check(self.lib.marl_ring_sample(self.handle, C.c_uint32(draw_index), C.c_int32(B), C.byref(sb)))
        return out

    def get_state(self) -> dict:
        s = StateView()
        _check(self.lib.marl_actor_get_state(self.handle, C.byref(s)))
        c = self.cfg
        E, n, H = c["E"], c["n"], c["H"]
        u8 = self.state_mem
        base = u8.data_ptr()

        def arr(ptr, dtype, shape):
            cnt = 1
            for x in shape:
                cnt *= x
            nb = torch.empty((), dtype=dtype).element_size() * cnt
            return u8[ptr - base: ptr - base + nb].view(dtype).view(shape)

        return dict(h=arr(s.h, torch.float32, (E, n, H)), last_action=arr(s.last_action, torch.int32, (E, n)),
                    slot=arr(s.slot, torch.int32, (E,)), pos=arr(s.pos, torch.int32, (E,)),
                    ep_count=arr(s.ep_count, torch.int64, (E,)), step=int(s.step))

    def set_state(self, st: dict):
        s = StateView(st["h"].data_ptr(), st["last_action"].data_ptr(), st["slot"].data_ptr(), st["pos"].data_ptr(),
                      st["ep_count"].data_ptr(), int(st["step"]))
        _check(self.lib.marl_actor_set_state(self.handle, C.byref(s)))

    def status(self):
        st = C.c_uint32(0)
        cn = Counters()
        _check(self.lib.marl_actor_status(self.handle, C.byref(st), C.byref(cn)))
        return int(st.value), {k: int(getattr(cn, k)) for k, _ in Counters._fields_}

    def reset(self):
        _check(self.lib.marl_actor_reset(self.handle))

    @property
    def kernel_name(self) -> str:
        return self.lib.marl_actor_kernel_name(self.handle).decode()

    @property
    def launch_count(self) -> int:
        return int(self.lib.marl_actor_launch_count(self.handle))

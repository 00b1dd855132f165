"""ctypes access to the CPU oracle (``marl_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, the smoke check and the benchmark's CPU-baseline
leg.  Nothing on the product path may import this package, and this package imports nothing from the
CUDA library.

The wrapper only marshals numpy arrays; every number is computed by the C++ file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "marl_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

CNT_STEPS, CNT_EPISODES, CNT_EXPLORE, CNT_NO_AVAIL, CNT_TRUNCATED, CNT_N = range(6)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-Wall", "-shared", "-fPIC", "-pthread",
             "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class Dims(C.Structure):
    _fields_ = [("n_envs", C.c_int32), ("n_agents", C.c_int32), ("obs_dim", C.c_int32),
                ("n_actions", C.c_int32), ("hidden", C.c_int32), ("ring_episodes", C.c_int32),
                ("ring_steps", C.c_int32), ("precision", C.c_int32), ("seed", C.c_uint64),
                ("n_types", C.c_int32), ("reserved", C.c_int32), ("agent_type", C.c_void_p)]


class Env(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("obs_law", C.c_int32), ("done_thresh24", C.c_uint32),
                ("avail_thresh_first", C.c_uint32), ("avail_thresh_rest", C.c_uint32),
                ("avail_split", C.c_int32), ("n_type0", C.c_int32), ("type_block_start", C.c_int32),
                ("type_block_len", C.c_int32)]


_P = C.c_void_p


class _Weights(C.Structure):
    _fields_ = [(k, _P) for k in ("W1", "b1", "W_ih", "b_ih", "W_hh", "b_hh", "W2", "b2")]


class _State(C.Structure):
    _fields_ = [(k, _P) for k in ("h", "last_action", "slot", "pos", "ep_count")]


class _Ring(C.Structure):
    _fields_ = [(k, _P) for k in ("obs", "avail", "action", "q", "reward", "done", "slot_epid",
                                  "slot_len", "slot_complete")]


class _Trace(C.Structure):
    _fields_ = [(k, _P) for k in ("obs", "avail", "reward", "done", "q", "h", "action", "action_free",
                                  "explore", "u", "slot", "pos")]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_bf16_round.restype = C.c_float
        _lib.oracle_bf16_round.argtypes = [C.c_float]
        _lib.oracle_uniform24.restype = C.c_float
        _lib.oracle_uniform24.argtypes = [C.c_uint32]
        _lib.oracle_eps_at.restype = C.c_float
        _lib.oracle_eps_at.argtypes = [C.c_double, C.c_double, C.c_int32, C.c_uint32]
        _lib.oracle_select_action.restype = C.c_int32
        _lib.oracle_hardware_threads.restype = C.c_int32
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(_P)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def make_dims(cfg: dict) -> Dims:
    """cfg uses the keys E, n, D, A, H, C, L, precision ('fp32'|'bf16' or 0|1), seed, and optionally agent_type
    (a list of n unit types: with more than one type the weights are a list of networks, one per type)."""
    prec = cfg["precision"]
    prec = {"fp32": 0, "bf16": 1}.get(prec, prec)
    d = Dims(cfg["E"], cfg["n"], cfg["D"], cfg["A"], cfg["H"], cfg["C"], cfg["L"], int(prec), int(cfg["seed"]),
             0, 0, None)
    types = cfg.get("agent_type")
    if types is not None:
        arr = np.ascontiguousarray(types, dtype=np.int32)
        assert arr.shape == (cfg["n"],) and arr.min() >= 0
        d._keep_types = arr                      # keeps the array alive as long as the struct
        d.n_types = int(arr.max()) + 1
        d.agent_type = arr.ctypes.data_as(C.c_void_p)
    return d


def make_env(env: dict) -> Env:
    return Env(int(env["seed"]), int(env["obs_law"]), int(env["done_thresh24"]),
               int(env["avail_thresh_first"]), int(env["avail_thresh_rest"]), int(env["avail_split"]),
               int(env["n_type0"]), int(env["type_block_start"]), int(env["type_block_len"]))


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().oracle_philox4x32_10(_ptr(ctr), _ptr(key), _ptr(out))
    return out


def bf16_round(x: float) -> float:
    return float(lib().oracle_bf16_round(C.c_float(x)))


def uniform24(w: int) -> float:
    return float(lib().oracle_uniform24(C.c_uint32(w)))


def eps_at(eps_start: float, eps_end: float, anneal_steps: int, t: int) -> float:
    return float(lib().oracle_eps_at(eps_start, eps_end, anneal_steps, t))


def hardware_threads() -> int:
    return int(lib().oracle_hardware_threads())


_WNAMES = ("W1", "b1", "W_ih", "b_ih", "W_hh", "b_hh", "W2", "b2")


def _weights_struct(w):
    """One network (a dict) or, for per-type networks, a list of them (an array of structs on the C side)."""
    if isinstance(w, dict):
        keep = {k: _c(w[k], np.float32) for k in _WNAMES}
        return _Weights(*[_ptr(keep[k]) for k in _WNAMES]), keep
    keep = [{k: _c(wk[k], np.float32) for k in _WNAMES} for wk in w]
    arr = (_Weights * len(keep))(*[_Weights(*[_ptr(kk[k]) for k in _WNAMES]) for kk in keep])
    return arr, keep


def env_emit(cfg: dict, env: dict, t: int, e: int):
    """Synthetic environment output of (step t, env e): obs [n][D], avail [n][A], reward, done."""
    d = make_dims(cfg)
    obs = np.zeros((cfg["n"], cfg["D"]), np.float32)
    avail = np.zeros((cfg["n"], cfg["A"]), np.uint8)
    reward = C.c_float(0)
    done = C.c_uint8(0)
    ev = make_env(env)
    lib().oracle_env_emit(C.byref(d), C.byref(ev), C.c_uint32(t), C.c_uint32(e), _ptr(obs), _ptr(avail),
                          C.byref(reward), C.byref(done))
    return obs, avail, float(reward.value), int(done.value)


def agent_forward(cfg: dict, w: dict, obs, agent: int, last_action: int, h_prev):
    """One row of the agent network: returns (q [A], h_new [H]) as float32."""
    d = make_dims(cfg)
    ws, keep = _weights_struct(w)
    obs = _c(obs, np.float32)
    h_prev = _c(h_prev, np.float32)
    q = np.zeros(cfg["A"], np.float32)
    h = np.zeros(cfg["H"], np.float32)
    lib().oracle_agent_forward(C.byref(d), C.byref(ws), _ptr(obs), C.c_int32(agent), C.c_int32(last_action),
                               _ptr(h_prev), _ptr(q), _ptr(h))
    del keep
    return q, h


def select_action(q, avail, eps: float, seed: int, t: int, e: int, i: int):
    """Returns (action, explore, u, no_avail)."""
    q = _c(q, np.float32)
    avail = _c(avail, np.uint8)
    ex = C.c_uint8(0)
    u = C.c_float(0)
    na = C.c_uint8(0)
    a = lib().oracle_select_action(_ptr(q), _ptr(avail), C.c_int32(len(q)), C.c_float(eps), C.c_uint64(seed),
                                   C.c_uint32(t), C.c_uint32(e), C.c_uint32(i), C.byref(ex), C.byref(u),
                                   C.byref(na))
    return int(a), int(ex.value), float(u.value), int(na.value)


def select_batch(q, avail, eps, seed: int, t, e, i):
    """Row-wise select_action: q [N][A], avail [N][A], eps/t/e/i [N] -> (action [N], explore [N])."""
    q = _c(q, np.float32)
    avail = _c(avail, np.uint8)
    N, A = q.shape
    eps = _c(np.broadcast_to(eps, (N,)), np.float32)
    t = _c(np.broadcast_to(t, (N,)), np.uint32)
    e = _c(np.broadcast_to(e, (N,)), np.uint32)
    i = _c(np.broadcast_to(i, (N,)), np.uint32)
    act = np.zeros(N, np.int32)
    ex = np.zeros(N, np.uint8)
    lib().oracle_select_batch(_ptr(q), _ptr(avail), C.c_int32(A), C.c_int64(N), _ptr(eps), C.c_uint64(seed),
                              _ptr(t), _ptr(e), _ptr(i), _ptr(act), _ptr(ex))
    return act, ex


@dataclass
class Session:
    """State, replay-pool image and counters of the oracle for a list of environments."""
    cfg: dict
    weights: dict
    env_ids: np.ndarray
    with_ring: bool = True
    n_threads: int = 1
    h: np.ndarray = field(init=False)
    last_action: np.ndarray = field(init=False)
    slot: np.ndarray = field(init=False)
    pos: np.ndarray = field(init=False)
    ep_count: np.ndarray = field(init=False)
    ring: dict = field(init=False)
    counters: np.ndarray = field(init=False)
    t: int = 0

    def __post_init__(self):
        c = self.cfg
        self.env_ids = _c(self.env_ids, np.int32)
        Es, n, D, A, H, L = len(self.env_ids), c["n"], c["D"], c["A"], c["H"], c["L"]
        assert c["C"] % c["E"] == 0
        S = c["C"] // c["E"]
        self.S = S
        self.h = np.zeros((Es, n, H), np.float32)
        self.last_action = np.zeros((Es, n), np.int32)
        self.slot = np.zeros(Es, np.int32)
        self.pos = np.zeros(Es, np.int32)
        self.ep_count = np.zeros(Es, np.int64)
        self.counters = np.zeros(CNT_N, np.uint64)
        if self.with_ring:
            self.ring = dict(
                obs=np.zeros((Es * S, L, n, D), np.float32), avail=np.zeros((Es * S, L, n, A), np.uint8),
                action=np.zeros((Es * S, L, n), np.int32), q=np.zeros((Es * S, L, n, A), np.float32),
                reward=np.zeros((Es * S, L), np.float32), done=np.zeros((Es * S, L), np.uint8),
                slot_epid=np.zeros(Es * S, np.int64), slot_len=np.zeros(Es * S, np.int32),
                slot_complete=np.zeros(Es * S, np.uint8))
        else:
            self.ring = None
        self._d = make_dims(c)
        self._w, self._wkeep = _weights_struct(self.weights)
        st, rg = self._structs()
        lib().oracle_init(C.byref(self._d), _ptr(self.env_ids), C.c_int32(Es), C.byref(st),
                          C.byref(rg) if rg is not None else None)

    def set_weights(self, weights: dict):
        """The shared model after a learner update (Sec. III-B): used by every later step."""
        self.weights = weights
        self._w, self._wkeep = _weights_struct(weights)

    def _structs(self):
        st = _State(_ptr(self.h), _ptr(self.last_action), _ptr(self.slot), _ptr(self.pos), _ptr(self.ep_count))
        rg = None
        if self.ring is not None:
            r = self.ring
            rg = _Ring(*[_ptr(r[k]) for k in ("obs", "avail", "action", "q", "reward", "done", "slot_epid",
                                              "slot_len", "slot_complete")])
        return st, rg

    def _alloc_trace(self, T, want, rows=None):
        c = self.cfg
        Es, n, D, A, H = (len(self.env_ids) if rows is None else rows), c["n"], c["D"], c["A"], c["H"]
        shapes = dict(obs=((T, Es, n, D), np.float32), avail=((T, Es, n, A), np.uint8),
                      reward=((T, Es), np.float32), done=((T, Es), np.uint8), q=((T, Es, n, A), np.float32),
                      h=((T, Es, n, H), np.float32), action=((T, Es, n), np.int32),
                      action_free=((T, Es, n), np.int32), explore=((T, Es, n), np.uint8),
                      u=((T, Es, n), np.float32), slot=((T, Es), np.int32), pos=((T, Es), np.int32))
        tr = {k: (np.zeros(*shapes[k]) if k in want else None) for k in shapes}
        ts = _Trace(*[_ptr(tr[k]) for k in ("obs", "avail", "reward", "done", "q", "h", "action", "action_free",
                                             "explore", "u", "slot", "pos")])
        return tr, ts

    ALL_TRACES = ("obs", "avail", "reward", "done", "q", "h", "action", "action_free", "explore", "u", "slot",
                  "pos")

    def rollout(self, env: dict, T: int, eps_start: float, eps_end: float = 0.0, anneal_steps: int = 0,
                adopt=None, trace=ALL_TRACES):
        """T steps against the synthetic environment from the session's step counter.  Returns traces."""
        Es = len(self.env_ids)
        tr, ts = self._alloc_trace(T, set(trace or ()))
        st, rg = self._structs()
        ev = make_env(env)
        if adopt is not None:
            adopt = _c(adopt, np.int32)
            assert adopt.shape == (T, Es, self.cfg["n"])
        lib().oracle_rollout(C.byref(self._d), C.byref(self._w), C.byref(ev), _ptr(self.env_ids), C.c_int32(Es),
                             C.c_uint32(self.t), C.c_int32(T), C.c_double(eps_start), C.c_double(eps_end),
                             C.c_int32(anneal_steps), _ptr(adopt), C.byref(st),
                             C.byref(rg) if rg is not None else None, C.byref(ts), _ptr(self.counters),
                             C.c_int32(self.n_threads))
        self.t += T
        return {k: v for k, v in tr.items() if v is not None}

    def step(self, obs, avail, reward, done, eps: float, adopt=None, trace=()):
        """One decision step on caller-supplied environment outputs.  Returns (actions, traces)."""
        c = self.cfg
        Es, n = len(self.env_ids), c["n"]
        obs = _c(obs, np.float32)
        avail = _c(avail, np.uint8)
        reward = _c(reward, np.float32)
        done = _c(done, np.uint8)
        assert obs.shape == (Es, n, c["D"]) and avail.shape == (Es, n, c["A"])
        if adopt is not None:
            adopt = _c(adopt, np.int32)
        tr, ts = self._alloc_trace(1, set(trace or ()))
        st, rg = self._structs()
        actions = np.zeros((Es, n), np.int32)
        lib().oracle_step(C.byref(self._d), C.byref(self._w), _ptr(self.env_ids), C.c_int32(Es),
                          C.c_uint32(self.t), C.c_float(eps), _ptr(obs), _ptr(avail), _ptr(reward), _ptr(done),
                          _ptr(adopt), C.byref(st), C.byref(rg) if rg is not None else None, _ptr(actions),
                          C.byref(ts), C.c_int32(0), _ptr(self.counters), C.c_int32(self.n_threads))
        self.t += 1
        return actions, {k: v[0] for k, v in tr.items() if v is not None}

    def step_lagged(self, env_ids, obs, avail, prev_reward, prev_done, eps: float, adopt=None, trace=()):
        """step_subset when the environment answers after the action (Algorithm 1: the reward of an action comes
        back with the next observation): prev_reward / prev_done belong to each environment's previous action."""
        return self.step_subset(env_ids, obs, avail, prev_reward, prev_done, eps, adopt=adopt, trace=trace,
                                lagged=True)

    def step_subset(self, env_ids, obs, avail, reward, done, eps: float, adopt=None, trace=(), lagged=False):
        """One decision step for the listed environments only (actors are asynchronous, Sec. III-A: the worker
        serves the observations that have arrived).  Index plumbing around the same step routine: the listed rows of
        the state and of the pool image are copied out, stepped with the session's step counter, and copied back;
        every other row is untouched.  Returns (actions [M][n], traces)."""
        c = self.cfg
        ids = _c(env_ids, np.int32)
        M, n, S = len(ids), c["n"], self.S
        where = {int(e): x for x, e in enumerate(self.env_ids)}
        loc = np.array([where[int(e)] for e in ids], np.int64)
        assert len(set(loc.tolist())) == M, "an environment is listed twice"
        obs = _c(obs, np.float32)
        avail = _c(avail, np.uint8)
        reward = _c(reward, np.float32)
        done = _c(done, np.uint8)
        assert obs.shape == (M, n, c["D"]) and avail.shape == (M, n, c["A"]) and reward.shape == (M,)
        if adopt is not None:
            adopt = _c(adopt, np.int32)
        sub = {k: np.ascontiguousarray(getattr(self, k)[loc]) for k in ("h", "last_action", "slot", "pos", "ep_count")}
        st = _State(*[_ptr(sub[k]) for k in ("h", "last_action", "slot", "pos", "ep_count")])
        rg, rsub = None, None
        if self.ring is not None:
            names = ("obs", "avail", "action", "q", "reward", "done", "slot_epid", "slot_len", "slot_complete")
            rows = (loc[:, None] * S + np.arange(S)[None, :]).reshape(-1)       # pool rows of the listed environments
            rsub = {k: np.ascontiguousarray(self.ring[k][rows]) for k in names}
            rg = _Ring(*[_ptr(rsub[k]) for k in names])
        tr, ts = self._alloc_trace(1, set(trace or ()), rows=M)
        actions = np.zeros((M, n), np.int32)
        if lagged:
            lib().oracle_step_lagged(C.byref(self._d), C.byref(self._w), _ptr(ids), C.c_int32(M), C.c_uint32(self.t),
                                     C.c_float(eps), _ptr(obs), _ptr(avail), _ptr(reward), _ptr(done), _ptr(adopt),
                                     C.byref(st), C.byref(rg) if rg is not None else None, _ptr(actions), C.byref(ts),
                                     _ptr(self.counters))
        else:
            lib().oracle_step(C.byref(self._d), C.byref(self._w), _ptr(ids), C.c_int32(M), C.c_uint32(self.t),
                              C.c_float(eps), _ptr(obs), _ptr(avail), _ptr(reward), _ptr(done), _ptr(adopt),
                              C.byref(st), C.byref(rg) if rg is not None else None, _ptr(actions), C.byref(ts),
                              C.c_int32(0), _ptr(self.counters), C.c_int32(self.n_threads))
        for k, v in sub.items():
            getattr(self, k)[loc] = v
        if rsub is not None:
            for k, v in rsub.items():
                self.ring[k][rows] = v
        self.t += 1
        return actions, {k: v[0] for k, v in tr.items() if v is not None}


TAG_SAMPLE = 5        # Philox stream tag of the learner's episode draws
SAMPLE_ATTEMPTS = 16  # draws per batch element before it is reported empty


def ring_sample(ring: dict, seed: int, draw_index: int, B: int) -> dict:
    """The learner's draw of B episodes from the replay pool (Algorithm 3: the learner draws a batch of B samples at
    random from the pool), written out plainly.

    The paper fixes neither the law nor the unit of a sample; the reading taken here: a sample is one complete
    episode, drawn uniformly and with replacement among the slots whose episode is closed.  Batch element b of
    draw number `draw_index` makes up to SAMPLE_ATTEMPTS attempts; attempt a takes word 0 of the Philox4x32-10
    block with counter (draw_index, b, a, TAG_SAMPLE) and key (seed lo, seed hi), proposes slot
    floor(w0 * C / 2^32) and accepts it if that slot's episode is complete (with at least one step).  An element
    whose attempts all fail is empty: slot -1, length 0.  The batch is dense, [B][L][...], steps at and beyond
    an episode's length are zero.

    `ring` holds the pool as arrays indexed [slot][step] (the layout of Session.ring).  Test infrastructure only.
    """
    C_, L = ring["obs"].shape[0], ring["obs"].shape[1]
    out = dict(slot=np.full(B, -1, np.int32), len=np.zeros(B, np.int32), epid=np.full(B, -1, np.int64))
    for k in ("obs", "avail", "action", "q", "reward", "done"):
        out[k] = np.zeros((B,) + ring[k].shape[1:], ring[k].dtype)
    key = (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    for b in range(B):
        for a in range(SAMPLE_ATTEMPTS):
            w0 = philox4x32_10((draw_index & 0xFFFFFFFF, b, a, TAG_SAMPLE), key)[0]
            s = (int(w0) * C_) >> 32
            if ring["slot_complete"][s] == 1 and ring["slot_len"][s] >= 1:
                n_steps = int(ring["slot_len"][s])
                out["slot"][b], out["len"][b], out["epid"][b] = s, n_steps, ring["slot_epid"][s]
                for k in ("obs", "avail", "action", "q", "reward", "done"):
                    out[k][b, :n_steps] = ring[k][s, :n_steps]
                break
    return out

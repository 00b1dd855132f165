"""Pins of the oracle's episode sampler (Algorithm 3: the learner draws B samples from the replay pool): the draw is
re-derived with a big-integer Philox, its law is checked statistically, and the gather against brute force."""
import numpy as np

import oracle
from test_oracle_pins import _philox_bigint as philox_ref  # big-integer Philox4x32-10, independent of the oracle


def _fake_ring(C=37, L=6, n=2, D=3, A=4, seed=1, p_complete=0.6):
    """A pool image with arbitrary contents: some slots complete with random lengths, some open, some unused."""
    rng = np.random.default_rng(seed)
    ring = dict(obs=rng.standard_normal((C, L, n, D)).astype(np.float32),
                avail=rng.integers(0, 2, (C, L, n, A)).astype(np.uint8),
                action=rng.integers(0, A, (C, L, n)).astype(np.int32),
                q=rng.standard_normal((C, L, n, A)).astype(np.float32),
                reward=rng.standard_normal((C, L)).astype(np.float32),
                done=rng.integers(0, 2, (C, L)).astype(np.uint8),
                slot_epid=rng.integers(0, 1000, C).astype(np.int64),
                slot_len=rng.integers(1, L + 1, C).astype(np.int32),
                slot_complete=(rng.random(C) < p_complete).astype(np.uint8))
    ring["slot_len"][::7] = 0                      # a complete flag with no step never qualifies
    return ring


def test_draw_follows_the_stated_philox_stream():
    ring = _fake_ring()
    C = ring["obs"].shape[0]
    seed, k, B = 0x1234567890ABCDEF, 9, 40
    out = oracle.ring_sample(ring, seed, k, B)
    key = (seed & 0xFFFFFFFF, seed >> 32)
    for b in range(B):
        want = -1
        for a in range(oracle.SAMPLE_ATTEMPTS):
            w0 = philox_ref((k, b, a, 5), key)[0]
            s = (w0 * C) >> 32
            if ring["slot_complete"][s] == 1 and ring["slot_len"][s] >= 1:
                want = s
                break
        assert out["slot"][b] == want


def test_only_complete_episodes_and_exact_gather():
    ring = _fake_ring(seed=3)
    out = oracle.ring_sample(ring, 77, 0, 64)
    L = ring["obs"].shape[1]
    for b in range(64):
        s = out["slot"][b]
        assert s >= 0 and ring["slot_complete"][s] == 1
        n_steps = ring["slot_len"][s]
        assert out["len"][b] == n_steps >= 1 and out["epid"][b] == ring["slot_epid"][s]
        for k in ("obs", "avail", "action", "q", "reward", "done"):
            for l in range(L):                     # brute force, step by step
                want = ring[k][s, l] if l < n_steps else np.zeros_like(ring[k][s, l])
                assert np.array_equal(out[k][b, l], want), (k, b, l)


def test_empty_pool_and_exhausted_attempts_give_empty_elements():
    ring = _fake_ring(seed=5)
    ring["slot_complete"][:] = 0
    out = oracle.ring_sample(ring, 1, 2, 8)
    assert (out["slot"] == -1).all() and (out["len"] == 0).all() and (out["epid"] == -1).all()
    assert not out["obs"].any() and not out["action"].any()
    # one eligible slot among 1000: an element finds it with probability 1 - (1 - 1/1000)^16 ~ 1.6 %
    big = _fake_ring(C=1000, L=2, seed=6)
    big["slot_complete"][:] = 0
    big["slot_complete"][123] = 1
    big["slot_len"][123] = 2
    out = oracle.ring_sample(big, 5, 0, 400)
    hit = out["slot"] == 123
    assert ((out["slot"] == -1) | hit).all() and 0 <= hit.sum() <= 25


def test_uniform_over_complete_slots_and_independent_of_batch_position():
    ring = _fake_ring(C=16, seed=8, p_complete=0.75)
    ring["slot_len"][:] = 3
    ok = np.nonzero(ring["slot_complete"] == 1)[0]
    counts = np.zeros(16)
    for k in range(40):
        out = oracle.ring_sample(ring, 99, k, 100)
        assert (out["slot"] >= 0).all()
        counts += np.bincount(out["slot"], minlength=16)
    assert counts[ring["slot_complete"] == 0].sum() == 0
    exp = 4000 / len(ok)
    chi2 = ((counts[ok] - exp) ** 2 / exp).sum()
    assert chi2 < 3.0 * len(ok) + 10                 # far beyond the 99.9th percentile only for a broken law
    # different draw numbers and seeds give different batches; the same ones the same batch
    a, b = oracle.ring_sample(ring, 99, 3, 50), oracle.ring_sample(ring, 99, 3, 50)
    assert np.array_equal(a["slot"], b["slot"])
    assert not np.array_equal(a["slot"], oracle.ring_sample(ring, 99, 4, 50)["slot"])
    assert not np.array_equal(a["slot"], oracle.ring_sample(ring, 98, 3, 50)["slot"])

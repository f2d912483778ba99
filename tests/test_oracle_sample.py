"""Pins for the oracle's Philox4x32-10 and integer-CDF categorical sampler."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


def test_philox_matches_triton_interpreter(xo):
    """Triton ships its own Philox4x32-10; its CPU interpreter evaluates it without a GPU."""
    pytest.importorskip("triton")
    env = dict(os.environ, TRITON_INTERPRET="1", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(HERE, "philox_triton_ref.py")],
                       capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    cases = json.loads(r.stdout.strip().splitlines()[-1])
    assert len(cases) >= 40
    for c in cases:
        seed = c["seed"]
        got = xo.philox4x32_10((seed & 0xFFFFFFFF, seed >> 32), c["counter"])
        assert got == c["out"], c


def test_philox_is_a_bijection_of_the_counter_low_bits(xo):
    """For a fixed key distinct counters give distinct blocks; words look uniform."""
    seen = set()
    bits = np.zeros(32)
    n = 4096
    for i in range(n):
        o = xo.philox4x32_10((7, 9), (i, 0, 0, 0))
        seen.add(tuple(o))
        bits += [(o[0] >> b) & 1 for b in range(32)]
    assert len(seen) == n
    assert np.all(np.abs(bits / n - 0.5) < 0.05)


def _r64(xo, seed, env, step):
    o = xo.philox4x32_10((seed & 0xFFFFFFFF, seed >> 32), (env, step & 0xFFFFFFFF, step >> 32, 0))
    return o[0] | (o[1] << 32)


def test_sampler_closed_forms(xo):
    Ne = 64
    # one-hot distribution: always that action
    p = np.zeros((Ne, 5), np.float32); p[:, 3] = 1.0
    assert np.all(xo.sample(p, 11, 0) == 3)
    # all-zero row: No-Op (last index)
    assert np.all(xo.sample(np.zeros((Ne, 5), np.float32), 11, 0) == 4)
    # two equal halves: action 0 iff the 64-bit draw is below 2^63
    p = np.zeros((Ne, 3), np.float32); p[:, 0] = 0.5; p[:, 2] = 0.5
    act = xo.sample(p, 0xABCDEF0123, 77)
    for e in range(Ne):
        assert act[e] == (0 if _r64(xo, 0xABCDEF0123, e, 77) < (1 << 63) else 2)
    # zero-probability entries are never drawn, whatever the draw
    p = np.tile(np.array([0, 0.25, 0, 0.75, 0], np.float32), (Ne, 1))
    for step in range(50):
        assert set(xo.sample(p, 3, step)) <= {1, 3}


def test_sampler_exact_integer_cdf(xo):
    """Python big integers restate floor(r*Q/2^64) and the prefix search exactly."""
    rng = np.random.default_rng(5)
    Ne, A1 = 32, 17
    p = rng.random((Ne, A1)).astype(np.float32)
    p[:, ::3] = 0
    p = (p / p.sum(axis=1, keepdims=True)).astype(np.float32)
    seed, step = (1 << 40) + 12345, (1 << 33) + 5
    act = xo.sample(p, seed, step)
    for e in range(Ne):
        q = [int(np.floor(float(v) * 4294967296.0)) for v in p[e]]
        t = (_r64(xo, seed, e, step) * sum(q)) >> 64
        run, want = 0, A1 - 1
        for a, qa in enumerate(q):
            run += qa
            if run > t:
                want = a
                break
        assert act[e] == want


def test_sampler_frequencies(xo):
    p = np.array([0.05, 0.0, 0.4, 0.25, 0.3], np.float32)
    Ne, steps = 512, 200
    counts = np.zeros(5)
    tile = np.tile(p, (Ne, 1))
    for s in range(steps):
        counts += np.bincount(xo.sample(tile, 99, s), minlength=5)
    n = Ne * steps
    assert counts[1] == 0
    nz = p > 0
    chi2 = (((counts[nz] - n * p[nz]) ** 2) / (n * p[nz])).sum()
    assert chi2 < 21.1          # 3 degrees of freedom, far tail (p ~ 1e-4)

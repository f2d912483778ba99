"""Pins for the oracle's seeded weight initialisation (the blob xrl_init_weights defines): layout, Xavier
bounds, the uniform law, and exact values rebuilt from Triton's own Philox4x32-10 words."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

from workloads import configs

HERE = os.path.dirname(os.path.abspath(__file__))
M = dict(T=40, S=8, H=64, K=4, L=2, Hm=48, Hm2=16, Dg=2, dtype="fp32", A_max=6)


def _bound(m, name, shape):
    if len(shape) == 2:
        return np.float32(np.sqrt(6.0 / (shape[0] + shape[1])))
    if name.startswith("a_"):
        return np.float32(np.sqrt(6.0 / (m["H"] // m["K"] + 1)))
    if name.endswith("w2"):
        return np.float32(np.sqrt(6.0 / (shape[0] + 1)))
    return np.float32(0.1)


def test_layout_bounds_and_uniform_law(xo):
    blob = xo.init_weights(M, 11)
    assert blob.dtype == np.float32 and len(blob) == configs.weight_count(M)
    off = 0
    for name, shape in configs.weight_layout(M):
        n = int(np.prod(shape))
        w = blob[off:off + n].astype(np.float64)
        off += n
        b = float(_bound(M, name, shape))
        assert np.all(np.abs(w) <= b), name                       # Xavier-uniform support
        # every value is b * (k 2^-23 - 1) for an integer k < 2^24, up to the one rounding of the product
        k = np.rint((w / b + 1.0) * 2.0 ** 23)
        assert np.all((k >= 0) & (k < 2 ** 24)), name
        assert np.allclose(w, b * (k * 2.0 ** -23 - 1.0), rtol=2e-7, atol=0), name
        if n >= 2000:                                             # textbook uniform: mean 0, variance b^2 / 3
            assert abs(w.mean()) < 4 * b / np.sqrt(3 * n), name
            assert abs(w.var() / (b * b / 3) - 1) < 0.1, name
            assert w.max() > 0.98 * b and w.min() < -0.98 * b, name
    assert off == len(blob)
    # reproducible from the seed, different seeds differ, a wider model keeps nothing of a narrower one's prefix rule
    assert np.array_equal(blob, xo.init_weights(M, 11))
    assert not np.array_equal(blob, xo.init_weights(M, 12))
    one_hidden = dict(M, Hm2=0)
    assert len(xo.init_weights(one_hidden, 11)) == configs.weight_count(one_hidden)


def test_values_follow_from_tritons_philox_words(xo):
    """Element i = b * ((w >> 8) 2^-23 - 1) with w the first word of Philox4x32-10(seed; (i, 0, 0, 1)): the words
    come from Triton's own generator under its CPU interpreter."""
    pytest.importorskip("triton")
    env = dict(os.environ, TRITON_INTERPRET="1", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, os.path.join(HERE, "philox_triton_ref.py")],
                       capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    cases = [c for c in json.loads(r.stdout.strip().splitlines()[-1]) if c["counter"][3] == 1]
    assert len(cases) == 16
    m = dict(M, H=512, K=8, L=1, Hm=64, Hm2=0)                    # W0 alone has (16 + 40) * 512 = 28,672 entries
    layout = configs.weight_layout(m)
    starts = np.cumsum([0] + [int(np.prod(s)) for _, s in layout])
    for seed in sorted({c["seed"] for c in cases}):
        blob = xo.init_weights(m, seed)
        checked = 0
        for c in cases:
            i = c["counter"][0]
            if c["seed"] != seed or i >= len(blob):
                continue
            t = int(np.searchsorted(starts, i, side="right")) - 1
            b = _bound(m, *layout[t])
            u = np.float32(c["out"][0] >> 8) * np.float32(2.0 ** -23) - np.float32(1.0)
            assert blob[i] == np.float32(b * u), (seed, i, layout[t][0])
            checked += 1
        assert checked >= 7


INIT_MUTATIONS = [
    ("counter word 3 left at the action draws' value", "uint32_t(i >> 32), 0u, 1u, w);", "uint32_t(i >> 32), 0u, 0u, w);"),
    ("Xavier bound from the fan-in alone", "return float(std::sqrt(6.0 / double(fan_in + fan_out)));",
     "return float(std::sqrt(6.0 / double(fan_in)));"),
    ("attention vectors scaled like a matrix of the whole width", "fill(H, xavier(d, 1)); fill(H, xavier(d, 1));",
     "fill(H, xavier(H, 1)); fill(H, xavier(H, 1));"),
    ("second word of the block instead of the first", "const float u = float(w[0] >> 8)", "const float u = float(w[1] >> 8)"),
    ("value head sized like the policy head", "const int64_t in = head == 0 ? H : 2 * H;\n    fill(in * Hm, xavier(in, Hm)); fill(Hm, bias);\n    if (Hm2 > 0) { fill(Hm * Hm2, xavier(Hm, Hm2)); fill(Hm2, bias); }\n    fill(last, xavier(last, 1)); fill(1, bias);\n  }\n  return off;",
     "const int64_t in = H;\n    fill(in * Hm, xavier(in, Hm)); fill(Hm, bias);\n    if (Hm2 > 0) { fill(Hm * Hm2, xavier(Hm, Hm2)); fill(Hm2, bias); }\n    fill(last, xavier(last, 1)); fill(1, bias);\n  }\n  return off;"),
]


@pytest.mark.parametrize("name,old,new", INIT_MUTATIONS, ids=[m[0] for m in INIT_MUTATIONS])
def test_planted_mistake_in_the_initialisation_is_caught(xo, tmp_path, name, old, new):
    from test_oracle_mutations import _build
    mutant = _build(tmp_path, name, old, new)
    mutant.xo_philox4x32_10.restype = None
    saved = xo._lib
    caught = False
    try:
        xo._lib = mutant
        for check in (test_layout_bounds_and_uniform_law, test_values_follow_from_tritons_philox_words):
            try:
                check(xo)
            except (AssertionError, ValueError):
                caught = True
                break
    finally:
        xo._lib = saved
    assert caught, f"mutation '{name}' went unnoticed"

"""Pins for the oracle's PPO objective (Section 3.3.4, Eq. 3-5), its hand-written gradient and the advantage
estimator.  The gradient is checked against central differences of J computed here, in numpy, from the
outputs of the oracle's forward pass (which has its own pins); the loss against closed forms."""
import numpy as np
import pytest

from workloads import configs, dags

M = dict(T=4, S=8, H=8, K=2, L=2, Hm=6, Dg=1, dtype="fp32", A_max=4)


def _batch(seed, m, envs=(3, 2), edge_attr=False):
    rng = dags.make_rng(seed)
    graphs, env_off = [], [0]
    for c in envs:
        for _ in range(c + 1):
            g = dags.random_dag(rng, int(rng.integers(3, 9)), m["T"], 8, False, window=4)
            if edge_attr:
                g["edge_attr"] = dags.tensor_shape_attributes(rng, len(g["edge_src"]), 8, False)
            graphs.append(g)
        env_off.append(len(graphs))
    b = dags.flatten(graphs, env_off, m["A_max"])
    b["mask"][0, 1] = 0                       # one masked candidate
    b["model"] = m
    return b


def _objective(m, blob, batch, action, logp_old, adv, ret, eps, c1, c2, xo):
    """J from the forward pass's probabilities and values, written out independently of the oracle's loss."""
    out = xo.forward(m, blob, batch)
    p, v = out["probs"], out["value"]
    ne = len(v)
    lc = lv = le = 0.0
    for e in range(ne):
        ratio = p[e, action[e]] / np.exp(logp_old[e])
        lc += -min(ratio * adv[e], np.clip(ratio, 1 - eps, 1 + eps) * adv[e])
        lv += (v[e] - ret[e]) ** 2
        q = p[e][p[e] > 0]
        le += float(np.sum(q * np.log(q)))
    return (lc + c1 * lv + c2 * le) / ne, lc / ne, lv / ne, le / ne


@pytest.mark.parametrize("variant", ["plain", "two hidden layers", "edge attributes", "both ways", "one layer"])
def test_gradient_matches_central_differences(xo, variant):
    m = dict(M)
    if variant == "two hidden layers":
        m["Hm2"] = 5
    if variant == "edge attributes":
        m["edge_attr"] = True
    if variant == "both ways":
        m["both_ways"] = True
    if variant == "one layer":
        m["L"] = 1; m["K"] = 1
    b = _batch(3, m, edge_attr=(variant == "edge attributes"))
    blob, _ = configs.make_weights(m, 41, readout_scale=0.3)
    blob = blob.astype(np.float32)
    st, packed = xo.pack(b)
    assert st == 0
    rng = np.random.default_rng(5)
    ne = len(b["env_off"]) - 1
    action = np.array([0, m["A_max"]], np.int32)          # a candidate in env 0, No-Op in env 1
    base = xo.forward(m, blob, b)
    # old log-probabilities around the current ones: one ratio inside the clipping range with positive
    # advantage (unclipped term active), one outside with the clipped term active (flat)
    logp_now = np.log(base["probs"][np.arange(ne), action])
    logp_old = logp_now - np.array([0.05, -0.5])
    adv = np.array([0.7, 1.3])
    ret = rng.normal(size=ne)
    eps, c1, c2 = 0.2, 0.5, 0.01
    got = xo.ppo_grad(m, blob, b, packed, action, logp_old, adv, ret, eps, c1, c2)
    J = _objective(m, blob, b, action, logp_old, adv, ret, eps, c1, c2, xo)
    np.testing.assert_allclose(got["loss"], J, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(got["logp"], logp_now, rtol=1e-12)
    delta = 2.0 ** -18            # small, so that hardly any ReLU changes side inside the step (at 2^-15 one did)
    num = np.zeros(len(blob))
    for k in range(len(blob)):
        wp = blob.copy(); wp[k] += np.float32(delta)
        wm = blob.copy(); wm[k] -= np.float32(delta)
        jp = _objective(m, wp, b, action, logp_old, adv, ret, eps, c1, c2, xo)[0]
        jm = _objective(m, wm, b, action, logp_old, adv, ret, eps, c1, c2, xo)[0]
        num[k] = (jp - jm) / (float(wp[k]) - float(wm[k]))      # the step the float32 blob really took
    scale = np.abs(num).max()
    assert scale > 1e-4
    bad = np.abs(got["grad"] - num) > 1e-5 * scale + 1e-4 * np.abs(num)
    assert not bad.any(), (np.flatnonzero(bad)[:10], got["grad"][bad][:5], num[bad][:5])
    # the clipped transition contributes nothing through the policy: its share of the gradient is the value
    # and entropy part only (checked by the differences above); every block of the blob is exercised
    names = [n for n, shp in configs.weight_layout(m) for _ in range(int(np.prod(shp)))]
    touched = {n for n, g in zip(names, got["grad"]) if g != 0.0}
    assert {"W0", "b0", "W1", "a_src1", "a_dst1", "b1", "Wg", "bg", "pW1", "pw2", "vW1", "vw2", "vb2"} <= touched      # (pb2 shifts every logit alike: zero gradient)


def test_loss_closed_forms(xo):
    m = dict(M)
    b = _batch(4, m)
    blob, _ = configs.make_weights(m, 42, readout_scale=0.3)
    st, packed = xo.pack(b)
    base = xo.forward(m, blob, b)
    ne = len(b["env_off"]) - 1
    action = np.array([2, 1], np.int32)
    logp_now = np.log(base["probs"][np.arange(ne), action])
    adv = np.array([0.4, -1.1])
    # ratio 1 and value target = value: L_clip = -mean(A), L_vf = 0
    got = xo.ppo_grad(m, blob, b, packed, action, logp_now, adv, base["value"], 0.2, 0.5, 0.0)
    assert abs(got["loss"][1] + adv.mean()) < 1e-13 and abs(got["loss"][2]) < 1e-20
    # ratio far above 1 + eps with positive advantage: clipped at (1 + eps) A, no policy gradient at all
    got = xo.ppo_grad(m, blob, b, packed, action, logp_now - 1.0, np.array([1.0, 1.0]), base["value"], 0.2, 0.0, 0.0)
    assert abs(got["loss"][1] + 1.2) < 1e-13 and np.all(got["grad"] == 0.0)
    # ... with negative advantage the unclipped term is the smaller one: L_clip = -e A
    got = xo.ppo_grad(m, blob, b, packed, action, logp_now - 1.0, np.array([-1.0, -1.0]), base["value"], 0.2, 0.0, 0.0)
    assert abs(got["loss"][1] - np.e) < 1e-12
    # zero policy weights: every valid action equally likely, entropy term = -log(#valid actions)
    _, W = configs.make_weights(m, 42, readout_scale=0.3)
    W["pw2"][:] = 0.0
    blob0 = configs.pack_weights(m, W)
    got = xo.ppo_grad(m, blob0, b, packed, action, logp_now, adv, base["value"], 0.2, 0.5, 1.0)
    nvalid = b["mask"].sum(axis=1) + 1
    assert abs(got["loss"][3] + np.mean(np.log(nvalid))) < 1e-13
    # an action that is masked out is rejected
    with pytest.raises(ValueError):
        xo.ppo_grad(m, blob, b, packed, np.array([1, 0], np.int32), logp_now, adv, base["value"])


def test_gae_closed_forms(xo):
    r = np.array([1.0, 2.0, 3.0]); v = np.array([0.5, 0.25, 0.125, 4.0])
    nd = np.zeros(3, np.uint8)
    # lambda = 0: one-step temporal differences
    adv, ret = xo.gae(r, v, nd, 0.9, 0.0)
    np.testing.assert_allclose(adv, r + 0.9 * v[1:] - v[:-1], rtol=1e-15)
    # lambda = 1: discounted return to the end plus the bootstrapped tail, minus the value
    adv, ret = xo.gae(r, v, nd, 0.9, 1.0)
    G = np.array([1 + 0.9 * 2 + 0.81 * 3 + 0.729 * 4, 2 + 0.9 * 3 + 0.81 * 4, 3 + 0.9 * 4])
    np.testing.assert_allclose(ret, G, rtol=1e-15)
    np.testing.assert_allclose(adv, G - v[:-1], rtol=1e-15)
    # an episode end cuts both the bootstrap and the accumulation
    adv, ret = xo.gae(r, v, np.array([0, 1, 0], np.uint8), 0.9, 1.0)
    np.testing.assert_allclose(ret, [1 + 0.9 * 2, 2.0, 3 + 0.9 * 4], rtol=1e-15)
    # general case against the textbook double sum
    rng = np.random.default_rng(0)
    T = 7
    r = rng.normal(size=T); v = rng.normal(size=T + 1)
    adv, _ = xo.gae(r, v, np.zeros(T, np.uint8), 0.95, 0.8)
    d = r + 0.95 * v[1:] - v[:-1]
    want = [sum((0.95 * 0.8) ** k * d[t + k] for k in range(T - t)) for t in range(T)]
    np.testing.assert_allclose(adv, want, rtol=1e-13)


def test_mirrored_mode_is_the_definition_for_fp32_and_close_to_it_for_bf16(xo):
    """The debugging mode that keeps Z and the layer outputs as a bf16 model stores them changes nothing for
    an fp32 model and moves a bf16 model's loss and gradient by rounding noise only."""
    for dtype in ("fp32", "bf16"):
        m = dict(M, dtype=dtype, H=16, K=2)
        b = _batch(7, m)
        blob, _ = configs.make_weights(m, 3, readout_scale=0.3)
        blob = blob.astype(np.float32)
        st, packed = xo.pack(b)
        assert st == 0
        action = np.array([0, m["A_max"]], np.int32)
        args = (m, blob, b, packed, action, np.array([-1.0, -0.7]), np.array([0.7, -1.3]), np.array([0.2, -0.4]))
        exact = xo.ppo_grad(*args)
        mir = xo.ppo_grad(*args, mirrored=True)
        if dtype == "fp32":
            assert np.array_equal(exact["grad"], mir["grad"]) and np.array_equal(exact["loss"], mir["loss"])
        else:
            assert not np.array_equal(exact["grad"], mir["grad"])
            np.testing.assert_allclose(mir["loss"], exact["loss"], rtol=2e-2, atol=1e-3)
            assert np.linalg.norm(mir["grad"] - exact["grad"]) <= 5e-2 * np.linalg.norm(exact["grad"])

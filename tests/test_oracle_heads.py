"""Pins for the oracle's policy / value heads and masked softmax (Sections 3.3.2, 3.3.3)."""
import numpy as np
import pytest

import dense_ref
from workloads import configs

M = dict(T=6, S=8, H=16, K=2, L=1, Hm=12, Dg=1, dtype="fp32", A_max=6)


def _setup(num_envs, cands, seed=0, A=6, Hm2=0):
    m = dict(M, A_max=A, Hm2=Hm2)
    blob, W = configs.make_weights(m, 30 + seed)
    rng = np.random.default_rng(seed)
    env_off = np.concatenate([[0], np.cumsum([c + 1 for c in cands])]).astype(np.int32)
    emb = rng.random((env_off[-1], m["H"])) * 2.0
    mask = np.zeros((num_envs, A), np.uint8)
    for e, c in enumerate(cands):
        mask[e, :c] = 1
    batch = {"env_off": env_off, "mask": mask}
    return m, blob, W, batch, emb


def _second(W, p):
    """The optional second hidden layer of head `p` as keyword arguments of dense_ref.mlp."""
    return dict(Wh=W[p + "Wh"], bh=W[p + "bh"]) if (p + "Wh") in W else {}


@pytest.mark.parametrize("Hm2", [0, 5])
def test_policy_matches_bruteforce_mlp_and_softmax(xo, Hm2):
    m, blob, W, batch, emb = _setup(2, [4, 6], Hm2=Hm2)
    batch["mask"][0, 1] = 0
    st, logits, probs, value = xo.policy_value(m, blob, batch, emb)
    assert st == 0
    A = m["A_max"]
    for e in range(2):
        cur = batch["env_off"][e]
        C = batch["env_off"][e + 1] - cur - 1
        ell = {}
        for a in range(C):
            if batch["mask"][e, a]:
                ell[a] = dense_ref.mlp(emb[cur + 1 + a], W["pW1"], W["pb1"], W["pw2"], W["pb2"], **_second(W, "p"))
        ell[A] = dense_ref.mlp(emb[cur], W["pW1"], W["pb1"], W["pw2"], W["pb2"], **_second(W, "p"))
        z = sum(np.exp(v) for v in ell.values())
        for a in range(A + 1):
            if a in ell:
                assert abs(probs[e, a] - np.exp(ell[a]) / z) < 1e-13
                assert abs(logits[e, a] - ell[a]) < 1e-12
            else:
                assert probs[e, a] == 0.0
        assert abs(probs[e].sum() - 1.0) < 1e-13
        assert probs[e, A] > 0
        # value: [current || mean of valid candidates] through the value MLP
        valid = [a for a in range(C) if batch["mask"][e, a]]
        u = np.concatenate([emb[cur], np.mean([emb[cur + 1 + a] for a in valid], axis=0)])
        assert abs(value[e] - dense_ref.mlp(u, W["vW1"], W["vb1"], W["vw2"], W["vb2"], **_second(W, "v"))) < 1e-12


def test_second_hidden_layer_reduces_to_one_layer_when_it_is_the_identity(xo):
    """Hidden sizes [Hm, Hm] with Wh = I, bh = 0: the first layer's outputs are >= 0, so the second
    layer passes them through and the heads equal the one-hidden-layer heads with the same w2, b2.
    With Wh = 0 the output is the constant w2 . ReLU(bh) + b2 whatever the input."""
    m1, blob1, W1, batch, emb = _setup(2, [3, 5], seed=4)
    Hm = m1["Hm"]
    m2 = dict(m1, Hm2=Hm)
    _, W2 = configs.make_weights(m2, 99)
    for k in W1:
        W2[k] = W1[k]
    for p in "pv":
        W2[p + "Wh"] = np.eye(Hm, dtype=np.float32)
        W2[p + "bh"] = np.zeros(Hm, np.float32)
    blob2 = np.concatenate([W2[n].ravel() for n, _ in configs.weight_layout(m2)]).astype(np.float32)
    _, lg1, p1, v1 = xo.policy_value(m1, blob1, batch, emb)
    _, lg2, p2, v2 = xo.policy_value(m2, blob2, batch, emb)
    np.testing.assert_allclose(lg2, lg1, rtol=0, atol=1e-13)
    np.testing.assert_allclose(p2, p1, rtol=0, atol=1e-15)
    np.testing.assert_allclose(v2, v1, rtol=0, atol=1e-13)
    for p in "pv":
        W2[p + "Wh"] = np.zeros((Hm, Hm), np.float32)
        W2[p + "bh"] = np.linspace(-1, 1, Hm).astype(np.float32)
    blob3 = np.concatenate([W2[n].ravel() for n, _ in configs.weight_layout(m2)]).astype(np.float32)
    _, lg3, p3, v3 = xo.policy_value(m2, blob3, batch, emb)
    const_p = float(np.maximum(W2["pbh"].astype(np.float64), 0) @ W2["pw2"].astype(np.float64) + W2["pb2"][0])
    const_v = float(np.maximum(W2["vbh"].astype(np.float64), 0) @ W2["vw2"].astype(np.float64) + W2["vb2"][0])
    assert np.all(np.abs(lg3[np.isfinite(lg3)] - const_p) < 1e-13)
    assert np.all(np.abs(v3 - const_v) < 1e-13)
    # equal logits: the valid actions and No-Op share the probability evenly
    for e, c in enumerate([3, 5]):
        np.testing.assert_allclose(p3[e][p3[e] > 0], 1.0 / (c + 1), rtol=1e-13)


def test_identical_candidates_and_permutation(xo):
    m, blob, W, batch, emb = _setup(1, [5], seed=1)
    emb[3] = emb[1]                       # candidates 0 and 2 identical
    _, _, p, v = xo.policy_value(m, blob, batch, emb)
    assert p[0, 0] == p[0, 2]
    perm = np.array([2, 4, 0, 1, 3])
    emb2 = emb.copy()
    emb2[1:6] = emb[1:6][perm]
    _, _, p2, v2 = xo.policy_value(m, blob, batch, emb2)
    np.testing.assert_allclose(p2[0, :5], p[0, :5][perm], rtol=1e-13)
    assert abs(p2[0, 6] - p[0, 6]) < 1e-15
    assert abs(v2[0] - v[0]) < 1e-12      # the candidate mean does not depend on order


def test_no_candidates_gives_noop(xo):
    m, blob, W, batch, emb = _setup(2, [0, 3], seed=2)
    _, _, p, v = xo.policy_value(m, blob, batch, emb)
    assert p[0, -1] == 1.0 and np.all(p[0, :-1] == 0.0)
    u = np.concatenate([emb[0], np.zeros(m["H"])])
    assert abs(v[0] - dense_ref.mlp(u, W["vW1"], W["vb1"], W["vw2"], W["vb2"])) < 1e-12
    # every candidate masked behaves the same way
    batch["mask"][1, :] = 0
    _, _, p, _ = xo.policy_value(m, blob, batch, emb)
    assert p[1, -1] == 1.0


def test_mask_beyond_candidates_is_rejected(xo):
    m, blob, W, batch, emb = _setup(1, [3], seed=3)
    batch["mask"][0, 4] = 1
    st, *_ = xo.policy_value(m, blob, batch, emb)
    assert st == 1


def test_two_candidate_value_by_hand(xo):
    m, blob, W, batch, emb = _setup(1, [2], seed=4)
    _, _, _, v = xo.policy_value(m, blob, batch, emb)
    mean = 0.5 * (emb[1] + emb[2])
    hid = np.maximum(np.concatenate([emb[0], mean]) @ W["vW1"].astype(np.float64) + W["vb1"], 0)
    assert abs(v[0] - (hid @ W["vw2"].astype(np.float64) + W["vb2"][0])) < 1e-12

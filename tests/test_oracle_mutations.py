"""The pins must be sharp: each plausible slip planted in a copy of the oracle (on the CPU, in a scratch
directory) has to make the dense brute-force comparison or a heads/pack check fail."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import dense_ref
from workloads import configs, dags

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "xrl_oracle.cpp")

MUTATIONS = [
    ("LeakyReLU slope", "return x > 0.0 ? x : 0.2 * x;", "return x > 0.0 ? x : 0.1 * x;"),
    ("half-scores swapped", "s_src[size_t(j) * K + k] + s_dst[size_t(i) * K + k]",
     "s_src[size_t(i) * K + k] + s_dst[size_t(j) * K + k]"),
    ("one-hot offset", "x[S + op[gi]] = 1.0;", "x[S + op[gi] + 1 < F0 ? S + op[gi] + 1 : S] = 1.0;"),
    ("layer bias dropped", "acc = relu(acc + double(w.b[l][c]));", "acc = relu(acc);"),
    ("self term dropped", "for (int t = 0; t <= deg; ++t) { al[t] = std::exp(sc[t] - mx); sum += al[t]; }",
     "for (int t = 0; t <= deg; ++t) { al[t] = (t < deg || deg == 0) ? std::exp(sc[t] - mx) : 0.0; sum += al[t]; }"),
    ("own shape block dropped", "x[S + T + s] = stored_input(m, shape[size_t(gi) * S + s]);", "x[S + T + s] = 0.0;"),
    ("edge aggregate takes the consumer's shape", ": shape[size_t(col[e]) * S + s]);",
     ": shape[size_t(gi) * S + s]);"),
    ("readout mean instead of sum", "for (int c = 0; c < m.Dg; ++c) u[H + c] = g_attr ? g_attr[c] : 0.0;",
     "for (int c = 0; c < H; ++c) u[c] /= double(n > 0 ? n : 1);\n  for (int c = 0; c < m.Dg; ++c) u[H + c] = g_attr ? g_attr[c] : 0.0;"),
    ("global attribute ignored", "u[H + c] = g_attr ? g_attr[c] : 0.0;", "u[H + c] = 0.0;"),
    ("bf16 truncation instead of rounding", "u += 0x7FFFu + lsb;", "u += 0u * lsb;"),
    ("edge attributes read in CSR slot order", "edge_attr ? edge_attr[size_t(eid[e]) * S + s]",
     "edge_attr ? edge_attr[size_t(e) * S + s]"),
    ("consumers listed under the wrong node", "nbl[col[e] - lo].push_back(i);", "nbl[i].push_back(col[e] - lo);"),
    ("second hidden layer without its ReLU", "out += relu(acc) * double(w2[c]);", "out += acc * double(w2[c]);"),
    ("second hidden layer's bias dropped", "double acc = double(bh[c]);", "double acc = 0.0;"),
    ("second hidden layer reads the first layer transposed", "acc += y1[k] * double(Wh[size_t(k) * hid2 + c]);",
     "acc += y1[k] * double(Wh[size_t(c) * hid + k]);"),
    ("input features of a bf16 model left unrounded",
     "double stored_input(const Model& m, float v) { return m.dtype == 1 ? round_bf16(v) : double(v); }",
     "double stored_input(const Model& m, float v) { return double(v); }"),
    ("masked candidates counted in the value head's mean", "if (mask[size_t(e) * A_max + a]) {\n        ++nv;",
     "{\n        ++nv;"),
]


def _build(tmp_path, name, old, new):
    src = open(SRC).read()
    assert old in src, f"mutation target for '{name}' not found: the oracle changed, update this test"
    path = tmp_path / "mut.cpp"
    path.write_text(src.replace(old, new))
    so = tmp_path / "libmut.so"
    subprocess.run(["g++", "-std=c++17", "-O1", "-fPIC", "-shared", "-fopenmp", "-o", str(so), str(path)], check=True)
    return ctypes.CDLL(str(so))


def _pins_hold(xo):
    """A condensed version of the brute-force pins; returns False as soon as one breaks."""
    for dtype in ("fp32", "bf16"):
        m = dict(T=6, S=8, H=16, K=2, L=2, Hm=8, Dg=2, dtype=dtype, A_max=4)
        _, W = configs.make_weights(m, 11)
        rng = dags.make_rng(5)
        # shape features off the bf16 grid: the bf16 model has to round them itself
        graphs = [dags.random_dag(rng, 12, 6, 8, False, window=6) for _ in range(4)]
        b = dags.flatten(graphs, [0, len(graphs)], 4)
        st, p = xo.pack(b)
        if st != 0:
            return False
        g0 = np.random.default_rng(1).normal(size=(len(graphs), 2))
        # weights that are not on the bf16 grid exercise the rounding of the stored matrices
        out = xo.encode(m, configs.pack_weights(m, W), b, p, g0=g0)
        for gi, g in enumerate(graphs):
            want = dense_ref.encode_graph(g, W, m, g0[gi])
            if not np.allclose(out["emb"][gi], want, rtol=1e-10, atol=1e-11):
                return False
    # consumers among the neighbours
    m = dict(T=6, S=8, H=16, K=2, L=2, Hm=8, Dg=1, dtype="fp32", A_max=4, both_ways=True)
    _, W = configs.make_weights(m, 23)
    rng = dags.make_rng(12)
    graphs = [dags.random_dag(rng, 12, 6, 8, False, window=6) for _ in range(3)]
    b = dags.flatten(graphs, [0, len(graphs)], 4)
    st, p = xo.pack(b)
    if st != 0:
        return False
    out = xo.encode(m, configs.pack_weights(m, W), b, p)
    for gi, g in enumerate(graphs):
        if not np.allclose(out["emb"][gi], dense_ref.encode_graph(g, W, m), rtol=1e-10, atol=1e-11):
            return False
    # attributes on the edges (off the bf16 grid for the bf16 model too), edge lists shuffled
    for dtype in ("fp32", "bf16"):
        m = dict(T=6, S=8, H=16, K=2, L=1, Hm=8, Dg=1, dtype=dtype, A_max=4)
        _, W = configs.make_weights(m, 19)
        rng = dags.make_rng(6)
        graphs = [dags.random_dag(rng, 12, 6, 8, False, window=6) for _ in range(3)]
        nrng = np.random.default_rng(8)
        for g in graphs:
            perm = nrng.permutation(len(g["edge_src"]))
            g["edge_src"], g["edge_dst"] = g["edge_src"][perm], g["edge_dst"][perm]
            g["edge_attr"] = dags.tensor_shape_attributes(rng, len(perm), 8, False)
        b = dags.flatten(graphs, [0, len(graphs)], 4)
        st, p = xo.pack(b)
        if st != 0:
            return False
        out = xo.encode(m, configs.pack_weights(m, W), b, p)
        for gi, g in enumerate(graphs):
            if not np.allclose(out["emb"][gi], dense_ref.encode_graph(g, W, m), rtol=1e-10, atol=1e-11):
                return False
    # heads with two hidden layers (widths 7 and 7) against the brute-force MLP, one candidate masked
    m = dict(T=6, S=8, H=16, K=2, L=0, Hm=7, Hm2=7, Dg=1, dtype="fp32", A_max=3)
    blob, W = configs.make_weights(m, 17)
    emb = np.random.default_rng(2).random((4, 16)) * 2.0
    hb = {"env_off": np.array([0, 4], np.int32), "mask": np.array([[1, 0, 1]], np.uint8)}
    st, logits, probs, value = xo.policy_value(m, blob, hb, emb)
    if st != 0:
        return False
    ell = [dense_ref.mlp(emb[g], W["pW1"], W["pb1"], W["pw2"], W["pb2"], W["pWh"], W["pbh"]) for g in (1, 3, 0)]
    if not np.allclose(logits[0, [0, 2, 3]], ell, rtol=1e-12, atol=1e-12):
        return False
    u = np.concatenate([emb[0], (emb[1] + emb[3]) / 2.0])
    if abs(value[0] - dense_ref.mlp(u, W["vW1"], W["vb1"], W["vw2"], W["vb2"], W["vWh"], W["vbh"])) > 1e-12:
        return False
    return True


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(xo, tmp_path, name, old, new):
    assert _pins_hold(xo), "the unmodified oracle must pass"
    mutant = _build(tmp_path, name, old, new)
    mutant.xo_philox4x32_10.restype = None
    saved = xo._lib
    try:
        xo._lib = mutant
        assert not _pins_hold(xo), f"mutation '{name}' went unnoticed"
    finally:
        xo._lib = saved


# ---- the reverse pass of the PPO objective: planted mistakes must break the finite-difference pin ----------
PPO_MUTATIONS = [
    ("softmax reverse pass without the mean term", "al[t] * (dal[t] - dot) * (e > 0.0 ? 1.0 : 0.2)",
     "al[t] * dal[t] * (e > 0.0 ? 1.0 : 0.2)"),
    ("LeakyReLU slope ignored in the reverse pass", "al[t] * (dal[t] - dot) * (e > 0.0 ? 1.0 : 0.2)",
     "al[t] * (dal[t] - dot)"),
    ("a_dst collects the producer-side score gradients", "gw.a_dst[l][cc] += ds_dst[size_t(i) * K + k] * zs;",
     "gw.a_dst[l][cc] += ds_src[size_t(i) * K + k] * zs;"),
    ("value loss derivative without its factor 2", "c1 * 2.0 * (v - ret[e]) * inv_ne", "c1 * (v - ret[e]) * inv_ne"),
    ("candidate mean not divided in the reverse pass", "+= du[H + c] / double(nv);", "+= du[H + c];"),
    ("entropy gradient with the wrong sign inside", "(std::log(pr[a]) - plogp);", "(std::log(pr[a]) + plogp);"),
    ("ReLU of Eq. 8 ignored in the reverse pass", "dpre[c] = tp.emb[c] > 0.0 ? demb[c] : 0.0;", "dpre[c] = demb[c];"),
    ("gathered rows receive unweighted gradients", "dz[size_t(j) * H + k * d + c] += al[t] * dp[c];",
     "dz[size_t(j) * H + k * d + c] += dp[c];"),
    ("clipped term treated as if it had a slope", "(t1 <= t2) ? -adv[e] * ratio * inv_ne : 0.0;",
     "-adv[e] * ratio * inv_ne;"),
]


def _ppo_pin_holds(xo):
    import test_oracle_ppo as tp
    m = dict(tp.M, Hm2=5)
    b = tp._batch(3, m)
    blob, _ = configs.make_weights(m, 41, readout_scale=0.3)
    blob = blob.astype(np.float32)
    st, packed = xo.pack(b)
    if st != 0:
        return False
    ne = len(b["env_off"]) - 1
    action = np.array([0, m["A_max"]], np.int32)
    base = xo.forward(m, blob, b)
    logp_now = np.log(base["probs"][np.arange(ne), action])
    logp_old = logp_now - np.array([0.05, 0.5])      # second transition: ratio above 1 + eps, clipped (flat)
    adv = np.array([0.7, 1.3]); ret = np.array([0.3, -0.8])
    args = (action, logp_old, adv, ret, 0.2, 0.5, 0.05)
    got = xo.ppo_grad(m, blob, b, packed, *args)
    J = tp._objective(m, blob, b, *args, xo)
    if not np.allclose(got["loss"], J, rtol=1e-11, atol=1e-12):
        return False
    delta = np.float32(2.0 ** -18)
    scale = np.abs(got["grad"]).max()
    for k in range(0, len(blob), 5):
        wp = blob.copy(); wp[k] += delta
        wm = blob.copy(); wm[k] -= delta
        num = (tp._objective(m, wp, b, *args, xo)[0] - tp._objective(m, wm, b, *args, xo)[0]) / (float(wp[k]) - float(wm[k]))
        if abs(got["grad"][k] - num) > 1e-5 * scale + 1e-4 * abs(num):
            return False
    return True


@pytest.mark.parametrize("name,old,new", PPO_MUTATIONS, ids=[m[0] for m in PPO_MUTATIONS])
def test_planted_mistake_in_the_reverse_pass_is_caught(xo, tmp_path, name, old, new):
    assert _ppo_pin_holds(xo), "the unmodified oracle must pass"
    mutant = _build(tmp_path, name, old, new)
    mutant.xo_philox4x32_10.restype = None
    saved = xo._lib
    try:
        xo._lib = mutant
        assert not _ppo_pin_holds(xo), f"mutation '{name}' went unnoticed"
    finally:
        xo._lib = saved

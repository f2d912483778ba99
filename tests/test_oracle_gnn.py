"""Pins for the oracle's encoder (Section 3.4, Eq. 6-8): dense brute force, closed forms,
invariants.  None of the expected values comes from the oracle itself."""
import numpy as np
import pytest

import dense_ref
from workloads import configs, dags

M_SMALL = dict(T=6, S=8, H=16, K=2, L=2, Hm=8, Dg=1, dtype="fp32", A_max=4)


def _tiny_graphs(seed, count=4, n=12, T=6):
    rng = dags.make_rng(seed)
    gs = [dags.random_dag(rng, n, T, 8, False, window=6) for _ in range(count)]
    # a graph with duplicate edges and a node of in-degree 5
    g = dags.random_dag(rng, n, T, 8, False, window=6)
    g["edge_src"] = np.concatenate([g["edge_src"], [0, 0, 1, 2, 3]]).astype(np.int32)
    g["edge_dst"] = np.concatenate([g["edge_dst"], [n - 1, n - 1, n - 1, n - 1, n - 1]]).astype(np.int32)
    return gs + [g]


def _run(xo, m, W, graphs, **kw):
    b = dags.flatten(graphs, [0, len(graphs)], m["A_max"])
    st, p = xo.pack(b)
    assert st == 0
    blob = configs.pack_weights(m, W)
    return b, p, xo.encode(m, blob, b, p, **kw)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_encoder_matches_dense_bruteforce(xo, dtype):
    m = dict(M_SMALL, dtype=dtype)
    _, W = configs.make_weights(m, 11)
    graphs = _tiny_graphs(5)
    if dtype == "bf16":
        for g in graphs:
            g["shape"] = dags.round_to_bf16_grid(g["shape"])
    b, p, out = _run(xo, m, W, graphs)
    for gi, g in enumerate(graphs):
        want = dense_ref.encode_graph(g, W, m)
        np.testing.assert_allclose(out["emb"][gi], want, rtol=1e-12, atol=1e-12)


def test_bf16_model_rounds_its_own_input_features(xo):
    """Section 3.3.2: shape features and edge attributes are tensor shapes divided by a constant, i.e.
    arbitrary reals.  A bf16 model stores them in bf16, so features given off the bf16 grid must be rounded
    (to nearest, ties to even) before Eq. 6 uses them: the dense restatement does its own rounding, the
    result differs from the unrounded one, and equals what on-grid copies of the same features give."""
    m = dict(M_SMALL, dtype="bf16")
    _, W = configs.make_weights(m, 11)
    graphs = _tiny_graphs(21)
    rng = np.random.default_rng(4)
    for g in graphs:
        g["shape"] = (g["shape"] + rng.uniform(1e-4, 3e-3, size=g["shape"].shape)).astype(np.float32)
        assert not np.array_equal(g["shape"], dags.round_to_bf16_grid(g["shape"]))
    _, _, out = _run(xo, m, W, graphs)
    on_grid = [dict(g, shape=dense_ref.bf16_round(g["shape"]).astype(np.float32)) for g in graphs]
    _, _, out_grid = _run(xo, m, W, on_grid)
    np.testing.assert_array_equal(out["emb"], out_grid["emb"])
    unrounded = dict(m, dtype="fp32")
    for gi, g in enumerate(graphs):
        want = dense_ref.encode_graph(g, W, m)
        np.testing.assert_allclose(out["emb"][gi], want, rtol=1e-12, atol=1e-12)
        W_r = dict(W, W0=dense_ref.bf16_round(W["W0"]), **{f"W{l}": dense_ref.bf16_round(W[f"W{l}"]) for l in (1, 2)})
        assert not np.allclose(want, dense_ref.encode_graph(g, W_r, unrounded), rtol=1e-9, atol=1e-12)
    # the same for attributes that live on the edges
    eg = [dict(g) for g in graphs]
    for g in eg:
        a = dags.tensor_shape_attributes(dags.make_rng(len(g["edge_src"])), len(g["edge_src"]), 8, False)
        g["edge_attr"] = (a + rng.uniform(1e-4, 3e-3, size=a.shape)).astype(np.float32)
    _, _, out_e = _run(xo, m, W, eg)
    for gi, g in enumerate(eg):
        np.testing.assert_allclose(out_e["emb"][gi], dense_ref.encode_graph(g, W, m), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_neighbourhood_both_ways_matches_dense_bruteforce(xo, dtype):
    """Eq. 7 with the consumers of a node among its neighbours: dense row softmax weighted by A + A^T + I
    (repeated edges count in both directions)."""
    m = dict(M_SMALL, dtype=dtype, both_ways=True)
    _, W = configs.make_weights(m, 15)
    graphs = _tiny_graphs(9)
    if dtype == "bf16":
        for g in graphs:
            g["shape"] = dags.round_to_bf16_grid(g["shape"])
    b, p, out = _run(xo, m, W, graphs)
    one_way = dict(m, both_ways=False)
    for gi, g in enumerate(graphs):
        want = dense_ref.encode_graph(g, W, m)
        np.testing.assert_allclose(out["emb"][gi], want, rtol=1e-12, atol=1e-12)
        assert not np.allclose(want, dense_ref.encode_graph(g, W, one_way))


def test_both_ways_on_a_symmetric_graph_doubles_the_multiplicities(xo):
    """If every edge j -> i comes with its reverse i -> j, reading the neighbourhood both ways only doubles
    every neighbour's multiplicity: the softmax then weighs neighbours 2 : 1 against the self term, which
    the one-way reading reproduces when each edge is listed twice."""
    m = dict(M_SMALL, L=1)
    _, W = configs.make_weights(m, 16)
    rng = dags.make_rng(10)
    g = dags.random_dag(rng, 10, 6, 8, False, window=5)
    sym = dict(g, edge_src=np.concatenate([g["edge_src"], g["edge_dst"]]).astype(np.int32),
               edge_dst=np.concatenate([g["edge_dst"], g["edge_src"]]).astype(np.int32))
    twice = dict(sym, edge_src=np.concatenate([sym["edge_src"]] * 2), edge_dst=np.concatenate([sym["edge_dst"]] * 2))
    # Eq. 6 sums over in-edges, so compare the attention layer alone: node features after layer 1 given equal h0
    # is not observable separately; instead zero W0's edge block so that Eq. 6 ignores the edges
    W = dict(W)
    W0 = W["W0"].copy(); W0[:8] = 0.0; W["W0"] = W0
    _, _, a = _run(xo, dict(m, both_ways=True), W, [sym])
    _, _, b2 = _run(xo, m, W, [twice])
    np.testing.assert_allclose(a["emb"], b2["emb"], rtol=1e-12, atol=1e-13)


def _shuffle_edges(rng, g):
    perm = rng.permutation(len(g["edge_src"]))
    return dict(g, edge_src=g["edge_src"][perm], edge_dst=g["edge_dst"][perm])


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_edge_attributes_match_dense_bruteforce(xo, dtype):
    """Section 3.3.2 as written: attributes live on the edges.  Edge lists in shuffled order (so that the CSR
    slots are a non-trivial permutation of the input edges), repeated edges, attributes that differ between
    the repeats; the expectation sums attributes straight from the input edge list."""
    m = dict(M_SMALL, dtype=dtype)
    _, W = configs.make_weights(m, 13)
    rng = np.random.default_rng(3)
    graphs = [_shuffle_edges(rng, g) for g in _tiny_graphs(7)]
    for g in graphs:
        g["edge_attr"] = dags.tensor_shape_attributes(dags.make_rng(len(g["edge_src"])), len(g["edge_src"]), 8, dtype == "bf16")
        if dtype == "bf16":
            g["shape"] = dags.round_to_bf16_grid(g["shape"])
    b, p, out = _run(xo, m, W, graphs)
    assert "edge_attr" in b
    for gi, g in enumerate(graphs):
        want = dense_ref.encode_graph(g, W, m)
        np.testing.assert_allclose(out["emb"][gi], want, rtol=1e-12, atol=1e-12)
        plain = dense_ref.encode_graph({k: v for k, v in g.items() if k != "edge_attr"}, W, m)
        assert not np.allclose(want, plain)          # the attributes matter


def test_edge_attributes_equal_to_the_producers_features_change_nothing(xo):
    """Edges that carry exactly their producer's shape features reproduce the node-feature reading bit
    for bit (same values added in the same order)."""
    m = dict(M_SMALL)
    _, W = configs.make_weights(m, 14)
    rng = np.random.default_rng(4)
    graphs = [_shuffle_edges(rng, g) for g in _tiny_graphs(8)]
    b, p, base = _run(xo, m, W, graphs)
    for g in graphs:
        g["edge_attr"] = g["shape"][g["edge_src"]]
    b2, p2, out = _run(xo, m, W, graphs)
    assert np.array_equal(out["emb"], base["emb"])


def test_each_stage_matches_dense_bruteforce(xo):
    m = dict(M_SMALL)
    _, W = configs.make_weights(m, 12)
    graphs = _tiny_graphs(6)
    no = np.concatenate([[0], np.cumsum([len(g["op"]) for g in graphs])])
    for layer in range(m["L"] + 1):
        _, p, out = _run(xo, m, W, graphs, dump_layer=layer, want_nodes=True, want_alpha=layer > 0)
        for gi, g in enumerate(graphs):
            h = dense_ref.node_update(g, W, m)
            alphas = None
            for l in range(1, layer + 1):
                h, alphas = dense_ref.gat_layer(g, h, W, l, m, return_alpha=True)
            np.testing.assert_allclose(out["nodes"][no[gi]:no[gi + 1]], h, rtol=1e-12, atol=1e-12)
            if layer > 0:
                # attention weights: rows sum to one, and agree with the dense softmax
                A = dense_ref.adjacency(g)
                for k in range(m["K"]):
                    for i in range(len(g["op"])):
                        gi_ = no[gi] + i
                        e0, e1 = p["rowptr"][gi_], p["rowptr"][gi_ + 1]
                        tot = out["alpha_edge"][e0:e1, k].sum() + out["alpha_self"][gi_, k]
                        assert abs(tot - 1.0) < 1e-12
                        # dense alpha holds the row total per producer (multi-edges merged)
                        per_src = {}
                        for t in range(e0, e1):
                            j = p["col"][t] - no[gi]
                            per_src[j] = per_src.get(j, 0.0) + out["alpha_edge"][t, k]
                        for j, v in per_src.items():
                            assert abs(v - alphas[k][i, j]) < 1e-12
                        assert abs(out["alpha_self"][gi_, k] - alphas[k][i, i]) < 1e-12
                        assert A[i].sum() == e1 - e0


def test_eq6_chain_and_star_closed_forms(xo):
    """Chain: the edge aggregate of node i is the shape of node i-1.  In-star with n equal
    leaves: the centre's aggregate is n times the leaf shape.  The one-hot product is a row
    lookup of W0."""
    m = dict(M_SMALL, L=0)
    _, W = configs.make_weights(m, 13)
    rng = np.random.default_rng(0)
    n = 7
    chain = {"op": rng.integers(0, 6, n).astype(np.int32),
             "shape": rng.random((n, 8)).astype(np.float32),
             "edge_src": np.arange(n - 1, dtype=np.int32), "edge_dst": np.arange(1, n, dtype=np.int32)}
    leaf = rng.random(8).astype(np.float32)
    star = {"op": rng.integers(0, 6, n).astype(np.int32),
            "shape": np.tile(leaf, (n, 1)),
            "edge_src": np.arange(n - 1, dtype=np.int32),
            "edge_dst": np.full(n - 1, n - 1, dtype=np.int32)}
    _, _, out = _run(xo, m, W, [chain, star], dump_layer=0, want_nodes=True)
    W0, b0 = W["W0"].astype(np.float64), W["b0"].astype(np.float64)
    S, T = 8, 6
    for i in range(n):
        ebar = chain["shape"][i - 1].astype(np.float64) if i > 0 else np.zeros(8)
        want = ebar @ W0[:S] + W0[S + chain["op"][i]] + chain["shape"][i].astype(np.float64) @ W0[S + T:] + b0
        np.testing.assert_allclose(out["nodes"][i], np.maximum(want, 0), rtol=1e-12, atol=1e-13)
    c = n + n - 1
    want = (n - 1) * leaf.astype(np.float64) @ W0[:S] + W0[S + star["op"][-1]] \
        + leaf.astype(np.float64) @ W0[S + T:] + b0
    np.testing.assert_allclose(out["nodes"][c], np.maximum(want, 0), rtol=1e-12, atol=1e-13)


def test_eq7_chain_softmax_is_logistic(xo):
    """On a chain every interior node attends to {i-1, i}: alpha = logistic(e_prev - e_self)."""
    m = dict(M_SMALL, L=1, K=1)
    _, W = configs.make_weights(m, 14)
    rng = np.random.default_rng(1)
    n = 6
    chain = {"op": rng.integers(0, 6, n).astype(np.int32),
             "shape": rng.random((n, 8)).astype(np.float32),
             "edge_src": np.arange(n - 1, dtype=np.int32), "edge_dst": np.arange(1, n, dtype=np.int32)}
    _, _, out = _run(xo, m, W, [chain], dump_layer=1, want_nodes=True, want_alpha=True)
    h0 = dense_ref.node_update(chain, W, m)
    Z = h0 @ W["W1"].astype(np.float64)
    ss = Z @ W["a_src1"].astype(np.float64)
    sd = Z @ W["a_dst1"].astype(np.float64)
    lrelu = lambda x: x if x > 0 else 0.2 * x
    b1 = W["b1"].astype(np.float64)
    # node 0 has no in-edges: h' = ReLU(Z_0 + b)
    np.testing.assert_allclose(out["nodes"][0], np.maximum(Z[0] + b1, 0), rtol=1e-12, atol=1e-13)
    assert abs(out["alpha_self"][0, 0] - 1.0) < 1e-15
    for i in range(1, n):
        a_prev = 1.0 / (1.0 + np.exp(-(lrelu(ss[i - 1] + sd[i]) - lrelu(ss[i] + sd[i]))))
        assert abs(out["alpha_edge"][i - 1, 0] - a_prev) < 1e-12
        want = np.maximum(a_prev * Z[i - 1] + (1 - a_prev) * Z[i] + b1, 0)
        np.testing.assert_allclose(out["nodes"][i], want, rtol=1e-11, atol=1e-12)


def test_eq7_zero_attention_is_mean_aggregation(xo):
    m = dict(M_SMALL, L=1)
    _, W = configs.make_weights(m, 15, zero_attention=True)
    graphs = _tiny_graphs(8)
    _, _, out = _run(xo, m, W, graphs, dump_layer=1, want_nodes=True)
    off = 0
    for g in graphs:
        n = len(g["op"])
        h0 = dense_ref.node_update(g, W, m)
        Z = h0 @ W["W1"].astype(np.float64)
        Mx = dense_ref.adjacency(g) + np.eye(n)
        want = np.maximum((Mx @ Z) / Mx.sum(axis=1, keepdims=True) + W["b1"].astype(np.float64), 0)
        np.testing.assert_allclose(out["nodes"][off:off + n], want, rtol=1e-12, atol=1e-13)
        off += n


def test_eq7_identical_nodes_ignore_topology(xo):
    """With the edge-aggregate rows of W0 zeroed and one op/shape for all nodes, every node has
    the same h0, so every attention layer reduces to ReLU(W^T h + b) whatever the edges."""
    m = dict(M_SMALL, L=2)
    _, W = configs.make_weights(m, 16)
    W["W0"][:8] = 0.0
    g = _tiny_graphs(9)[-1]
    g["op"][:] = 3
    g["shape"][:] = g["shape"][0]
    _, _, out = _run(xo, m, W, [g], dump_layer=2, want_nodes=True)
    x = np.concatenate([np.zeros(8), np.eye(6)[3], g["shape"][0].astype(np.float64)])
    h = np.maximum(x @ W["W0"].astype(np.float64) + W["b0"], 0)
    for l in (1, 2):
        h = np.maximum(h @ W[f"W{l}"].astype(np.float64) + W[f"b{l}"], 0)
    for i in range(len(g["op"])):
        np.testing.assert_allclose(out["nodes"][i], h, rtol=1e-12, atol=1e-13)


def test_eq7_out_star_leaves_agree_and_heads_repeat(xo):
    rng = np.random.default_rng(2)
    n = 6
    star = {"op": np.full(n, 2, np.int32), "shape": np.tile(rng.random(8).astype(np.float32), (n, 1)),
            "edge_src": np.zeros(n - 1, np.int32), "edge_dst": np.arange(1, n, dtype=np.int32)}
    star["shape"][0] = rng.random(8)
    m1 = dict(M_SMALL, L=1, K=1, H=8)
    _, W1 = configs.make_weights(m1, 17)
    _, _, o1 = _run(xo, m1, W1, [star], dump_layer=1, want_nodes=True)
    for i in range(2, n):
        np.testing.assert_allclose(o1["nodes"][i], o1["nodes"][1], rtol=0, atol=0)
    # two heads whose blocks repeat the single head: output = the single head's, twice
    m2 = dict(M_SMALL, L=1, K=2, H=16)
    _, W2 = configs.make_weights(m2, 18)
    W2["W0"] = np.concatenate([W1["W0"], W1["W0"]], axis=1)
    W2["b0"] = np.concatenate([W1["b0"], W1["b0"]])
    blk = np.zeros((16, 16), np.float32)
    blk[:8, :8] = W1["W1"]; blk[:8, 8:] = W1["W1"]
    W2["W1"] = blk
    for k in ("a_src1", "a_dst1", "b1"):
        W2[k] = np.concatenate([W1[k], W1[k]])
    _, _, o2 = _run(xo, m2, W2, [star], dump_layer=1, want_nodes=True)
    np.testing.assert_allclose(o2["nodes"][:, :8], o1["nodes"], rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(o2["nodes"][:, 8:], o1["nodes"], rtol=1e-13, atol=1e-14)


def test_eq8_isolated_identical_nodes_and_global_attribute(xo):
    m = dict(M_SMALL, L=1, Dg=2)
    _, W = configs.make_weights(m, 19)
    n = 9
    g = {"op": np.full(n, 1, np.int32), "shape": np.tile(np.linspace(0, 1, 8, dtype=np.float32), (n, 1)),
         "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)}
    g0 = np.array([[0.7, -1.3]])
    _, _, out = _run(xo, m, W, [g], g0=g0)
    x = np.concatenate([np.zeros(8), np.eye(6)[1], g["shape"][0].astype(np.float64)])
    h = np.maximum(x @ W["W0"].astype(np.float64) + W["b0"], 0)
    h = np.maximum(h @ W["W1"].astype(np.float64) + W["b1"], 0)
    u = np.concatenate([n * h, g0[0]])
    want = np.maximum(u @ W["Wg"].astype(np.float64) + W["bg"], 0)
    np.testing.assert_allclose(out["emb"][0], want, rtol=1e-12, atol=1e-13)


def test_node_order_permutation_invariance(xo):
    m = dict(configs.MODEL[1])
    blob, W = configs.make_weights(m, 20)
    rng = np.random.default_rng(3)
    g = dags.random_dag(dags.make_rng(21), 64)
    perm = rng.permutation(64).astype(np.int32)        # old -> new
    inv = np.argsort(perm)
    g2 = {"op": g["op"][inv], "shape": g["shape"][inv],
          "edge_src": perm[g["edge_src"]], "edge_dst": perm[g["edge_dst"]]}
    _, _, o = _run(xo, m, W, [g, g2])
    np.testing.assert_allclose(o["emb"][0], o["emb"][1], rtol=1e-12, atol=1e-13)
    # permuting graphs permutes the rows of the embedding matrix
    _, _, o2 = _run(xo, m, W, [g2, g])
    np.testing.assert_array_equal(o2["emb"][::-1], o["emb"])


def test_mirrored_mode_stays_close_to_exact(xo):
    b = configs.make_batch(3, candidates=3)
    m = b["model"]
    blob, _ = configs.make_weights(m, 22, readout_scale=1.0 / 1200)
    _, p = xo.pack(b)
    e0 = xo.encode(m, blob, b, p, mode=0)["emb"]
    e1 = xo.encode(m, blob, b, p, mode=1)["emb"]
    assert np.all(np.abs(e0 - e1) <= 2e-2 + 2e-2 * np.abs(e0))
    assert np.abs(e0 - e1).max() > 0          # the rounding really happened

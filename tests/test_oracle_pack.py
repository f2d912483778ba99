"""Pins for the oracle's meta-graph packer (Section 3.3.2): brute-force reconstruction."""
import collections

import numpy as np

from workloads import configs, dags


def _check_against_input(batch, packed):
    B = batch["num_graphs"]
    no, eo = packed["node_off"], packed["edge_off"]
    # offsets are the prefix sums of the counts (closed form)
    assert np.array_equal(no, np.concatenate([[0], np.cumsum(batch["n_nodes"])]))
    assert np.array_equal(eo, np.concatenate([[0], np.cumsum(batch["n_edges"])]))
    rowptr, col, seg = packed["rowptr"], packed["col"], packed["seg_id"]
    assert rowptr[0] == 0 and rowptr[-1] == eo[-1]
    assert np.all(np.diff(rowptr) >= 0)
    assert np.all(np.diff(seg) >= 0)
    for g in range(B):
        assert np.all(seg[no[g]:no[g + 1]] == g)
    # per consumer, producers in the order of the input edge list
    want = collections.defaultdict(list)
    for g, gr in enumerate(dags.split(batch)):
        for s, d in zip(gr["edge_src"], gr["edge_dst"]):
            want[int(no[g] + d)].append(int(no[g] + s))
    for i in range(no[-1]):
        assert list(col[rowptr[i]:rowptr[i + 1]]) == want.get(i, []), i
    # eid: the input edge sitting in each CSR slot - a permutation of the edges that agrees with col, with
    # the row it sits in, and increases inside a row (input order kept)
    eid = packed["eid"]
    assert sorted(eid.tolist()) == list(range(int(eo[-1])))
    g_of_edge = np.repeat(np.arange(B), batch["n_edges"])
    for i in range(no[-1]):
        ks = np.arange(rowptr[i], rowptr[i + 1])
        es = eid[ks]
        assert np.all(np.diff(es) > 0)
        assert np.all(no[g_of_edge[es]] + batch["edge_dst"][es] == i)
        assert np.array_equal(col[ks], no[g_of_edge[es]] + batch["edge_src"][es])
    # env -> graph map
    for e in range(len(batch["env_off"]) - 1):
        assert np.all(packed["graph_env"][batch["env_off"][e]:batch["env_off"][e + 1]] == e)


def test_pack_bruteforce_cfg1(xo):
    b = configs.make_batch(1)
    st, p = xo.pack(b)
    assert st == 0
    _check_against_input(b, p)


def test_pack_bruteforce_rewrites_and_shuffled_edges(xo):
    b = configs.make_batch(2, candidates=5)
    rng = np.random.default_rng(0)
    # shuffle each graph's edge list: rows must follow the shuffled order
    eo = np.concatenate([[0], np.cumsum(b["n_edges"])])
    for g in range(b["num_graphs"]):
        perm = rng.permutation(eo[g + 1] - eo[g]) + eo[g]
        b["edge_src"][eo[g]:eo[g + 1]] = b["edge_src"][perm]
        b["edge_dst"][eo[g]:eo[g + 1]] = b["edge_dst"][perm]
    st, p = xo.pack(b)
    assert st == 0
    _check_against_input(b, p)


def test_pack_duplicates_isolated_and_empty(xo):
    g0 = {"op": np.zeros(4, np.int32), "shape": np.zeros((4, 8), np.float32),
          "edge_src": np.array([0, 0, 2, 0], np.int32), "edge_dst": np.array([3, 3, 3, 1], np.int32)}
    g1 = {"op": np.zeros(0, np.int32), "shape": np.zeros((0, 8), np.float32),
          "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)}
    g2 = {"op": np.zeros(2, np.int32), "shape": np.zeros((2, 8), np.float32),
          "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)}
    b = dags.flatten([g0, g1, g2], [0, 3], 4)
    st, p = xo.pack(b)
    assert st == 0
    assert list(p["rowptr"]) == [0, 0, 1, 1, 4, 4, 4]
    assert list(p["col"]) == [0, 0, 0, 2]
    assert list(p["node_off"]) == [0, 4, 4, 6]
    _check_against_input(b, p)


def test_pack_rejects_bad_graphs(xo):
    base = dags.random_dag(dags.make_rng(3), 16)
    for bad_src, bad_dst in [(5, 5), (16, 2), (-1, 2), (2, 16)]:
        g = {k: v.copy() for k, v in base.items()}
        g["edge_src"][0], g["edge_dst"][0] = bad_src, bad_dst
        st, _ = xo.pack(dags.flatten([g], [0, 1], 1))
        assert st == 2


def test_pack_relabel_roundtrip(xo):
    """Renumbering a graph's nodes permutes rows but keeps each row's producer multiset."""
    rng = np.random.default_rng(1)
    g = dags.random_dag(dags.make_rng(7), 40)
    perm = rng.permutation(40).astype(np.int32)      # old id -> new id
    g2 = {"op": np.zeros(40, np.int32), "shape": np.zeros((40, 8), np.float32),
          "edge_src": perm[g["edge_src"]], "edge_dst": perm[g["edge_dst"]]}
    _, p1 = xo.pack(dags.flatten([g], [0, 1], 1))
    _, p2 = xo.pack(dags.flatten([g2], [0, 1], 1))
    for i in range(40):
        a = sorted(perm[p1["col"][p1["rowptr"][i]:p1["rowptr"][i + 1]]])
        j = perm[i]
        assert a == sorted(p2["col"][p2["rowptr"][j]:p2["rowptr"][j + 1]])

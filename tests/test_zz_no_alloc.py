"""xrl_pack_csr_static: the packer for programs that must not allocate GPU memory at run time
(a server whose pool owns the whole device, a latency-bound loop that cannot afford cudaMalloc's
device-wide synchronisation).  It keeps its scratch in a fixed array inside the library, so these tests
pre-allocate every input and output, call it several times in a row on different batches (each call
finds the previous call's leftovers in the shared scratch) and require the same packed arrays, bit for
bit, as the regular xrl_pack_flat entry point and as the CPU oracle's packer.  One test uses graphs small
enough for the one-CTA-per-graph kernel (which touches only the count words of the scratch), the other
graphs too large for it, so that the in-degree counters, row cursors, unsorted edge slots, long-row list
and coarse edge table of the scratch are all written, left dirty and reused.  Collected last on purpose."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util

pytestmark = pytest.mark.gpu

KEYS = ("node_off", "edge_off", "seg_id", "graph_env", "rowptr", "col")


def _regular(batch):
    import paper_2304_14698_b200 as xrl
    ag = gpu_util.make_agent(batch)
    try:
        ag.pack(batch)
        out = xrl.xrl_batch_export(ag.batch)
        assert ag.device_status() == 0
        return out
    finally:
        ag.close()


def _static(batch, bufs):
    import torch
    import paper_2304_14698_b200 as xrl
    N, E, B = int(batch["n_nodes"].sum()), int(batch["n_edges"].sum()), batch["num_graphs"]
    bufs["op"][:N].copy_(torch.from_numpy(batch["op"]))
    bufs["edge_src"][:E].copy_(torch.from_numpy(batch["edge_src"]))
    bufs["edge_dst"][:E].copy_(torch.from_numpy(batch["edge_dst"]))
    for k in KEYS + ("status",):
        bufs[k].fill_(-7)                       # stale outputs must not survive
    xrl.xrl_pack_csr_static(0, batch["model"]["T"], batch["n_nodes"], batch["n_edges"], bufs["op"],
                            bufs["edge_src"], bufs["edge_dst"], batch["env_off"], bufs["node_off"],
                            bufs["edge_off"], bufs["seg_id"], bufs["graph_env"], bufs["rowptr"],
                            bufs["col"], bufs["status"])
    torch.cuda.synchronize()
    size = {"node_off": B + 1, "edge_off": B + 1, "seg_id": N, "graph_env": B, "rowptr": N + 1, "col": E}
    return {k: bufs[k][:size[k]].cpu().numpy() for k in KEYS}, int(bufs["status"].cpu()[0])


def _buffers():
    import torch
    cap_n, cap_e, cap_b = 131072, 524288, 4096
    i32 = dict(dtype=torch.int32, device="cuda")
    return {"op": torch.zeros(cap_n, **i32), "edge_src": torch.zeros(cap_e, **i32),
            "edge_dst": torch.zeros(cap_e, **i32), "node_off": torch.zeros(cap_b + 1, **i32),
            "edge_off": torch.zeros(cap_b + 1, **i32), "seg_id": torch.zeros(cap_n, **i32),
            "graph_env": torch.zeros(cap_b, **i32), "rowptr": torch.zeros(cap_n + 1, **i32),
            "col": torch.zeros(cap_e, **i32), "status": torch.zeros(1, **i32)}


def _oversized_batch(seed, n_big, long_rows):
    """A batch whose largest graph (n_big > 16,384 nodes) does not fit the one-CTA-per-graph kernel, next
    to a few small graphs and an empty one; some consumers of the large graph have far more than 32
    producers (repeats included); every edge list is shuffled."""
    rng = dags.make_rng(seed)
    nrng = np.random.default_rng(seed)
    big = dags.random_dag(rng, n_big, 32, 8, False, window=24)
    src, dst = [big["edge_src"]], [big["edge_dst"]]
    for k, count in enumerate(long_rows):
        consumer = n_big - 1 - 7 * k
        src.append(nrng.integers(0, consumer, count).astype(np.int32))
        dst.append(np.full(count, consumer, np.int32))
    big["edge_src"], big["edge_dst"] = np.concatenate(src), np.concatenate(dst)
    empty = {"op": np.zeros(0, np.int32), "shape": np.zeros((0, 8), np.float32),
             "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)}
    graphs = [dags.random_dag(rng, 300, 32, 8, False), big, empty, dags.random_dag(rng, 64, 32, 8, False),
              dags.random_dag(rng, 1500, 32, 8, False, window=40)]
    for g in graphs:
        perm = nrng.permutation(len(g["edge_src"]))
        g["edge_src"], g["edge_dst"] = g["edge_src"][perm], g["edge_dst"][perm]
    b = dags.flatten(graphs, [0, 3, 5], 4)
    b["model"] = dict(configs.MODEL[1], A_max=4)
    return b


def test_static_pack_of_graphs_too_large_for_one_cta_back_to_back(xo):
    """The path through global-memory counters: every region of the built-in scratch is used, and the next
    call (a different batch, then a malformed one, then the first again) starts from what the last left."""
    first = _oversized_batch(1, 20000, [40, 33, 600])
    second = _oversized_batch(2, 17500, [2000, 35])
    assert int(first["n_nodes"].max()) > 16384 and int(second["n_nodes"].max()) > 16384
    bufs = _buffers()
    for batch in (first, second, first):
        st, want = xo.pack(batch)
        assert st == 0
        assert int(np.diff(want["rowptr"]).max()) > 32          # rows beyond the one-thread ordering path
        ref = _regular(batch)
        got, status = _static(batch, bufs)
        assert status == 0
        for k in KEYS:
            assert np.array_equal(got[k], want[k]), ("oracle", k)
            assert np.array_equal(got[k], ref[k]), ("xrl_pack_flat", k)

    # a malformed large graph (an edge whose producer is its consumer) is reported, and the scratch it
    # leaves behind does not disturb the next, clean call
    bad = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in second.items()}
    e_big = int(bad["n_edges"][0]) + 11                          # an edge of the large graph
    bad["edge_src"][e_big] = bad["edge_dst"][e_big]
    _, status = _static(bad, bufs)
    assert status == 2
    st, want = xo.pack(second)
    got, status = _static(second, bufs)
    assert status == 0
    for k in KEYS:
        assert np.array_equal(got[k], want[k]), k


def test_static_pack_matches_regular_pack_twice_in_a_row(xo):
    import torch
    import paper_2304_14698_b200 as xrl
    first = configs.make_batch(2, candidates=40)              # ~23 k nodes, transformer-shaped
    second = configs.make_batch(4, candidates=20, seed=9)     # ~84 k nodes, rows of up to ~20 producers
    rng = np.random.default_rng(0)                            # shuffled edge lists: order must be restored
    perm = rng.permutation(int(second["n_edges"][0]))
    second["edge_src"][:len(perm)] = second["edge_src"][:len(perm)][perm]
    second["edge_dst"][:len(perm)] = second["edge_dst"][:len(perm)][perm]
    want = [_regular(first), _regular(second)]

    bufs = _buffers()
    for batch, ref in zip([first, second], want):
        got, status = _static(batch, bufs)
        assert status == 0
        st, oracle = xo.pack(batch)
        assert st == 0
        for k in KEYS:
            assert np.array_equal(got[k], ref[k]), k
            assert np.array_equal(got[k], oracle[k]), ("oracle", k)

    # a malformed graph is reported through the caller's status word, not by a fault
    bad = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in first.items()}
    bad["edge_src"][5] = bad["edge_dst"][5]
    _, status = _static(bad, bufs)
    assert status == 2
    # and a clean call afterwards is clean again
    got, status = _static(first, bufs)
    assert status == 0 and np.array_equal(got["col"], want[0]["col"])

    # sizes beyond the built-in scratch are refused up front
    big = configs.make_batch(4, candidates=40)               # ~164 k nodes > 131072
    with pytest.raises(xrl.XrlError) as e:
        xrl.xrl_pack_csr_static(0, 64, big["n_nodes"], big["n_edges"], bufs["op"], bufs["edge_src"],
                                bufs["edge_dst"], big["env_off"], bufs["node_off"], bufs["edge_off"],
                                bufs["seg_id"], bufs["graph_env"], bufs["rowptr"], bufs["col"], bufs["status"])
    assert e.value.status == 3

"""xrl_pack_csr_static: the packer for programs that must not allocate GPU memory at run time
(a server whose pool owns the whole device, a latency-bound loop that cannot afford cudaMalloc's
device-wide synchronisation).  It keeps its scratch in a fixed array inside the library, so this test
pre-allocates every input and output, calls it twice in a row on different batches (the second call
finds the first call's leftovers in the shared scratch) and requires the same packed arrays, bit for
bit, as the regular xrl_pack_flat entry point.  Collected last on purpose."""
import numpy as np
import pytest

from workloads import configs
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


def test_static_pack_matches_regular_pack_twice_in_a_row():
    import torch
    import paper_2304_14698_b200 as xrl
    first = configs.make_batch(2, candidates=40)              # ~23 k nodes, transformer-shaped
    second = configs.make_batch(4, candidates=20, seed=9)     # ~84 k nodes, rows of up to ~20 producers
    rng = np.random.default_rng(0)                            # shuffled edge lists: order must be restored
    perm = rng.permutation(int(second["n_edges"][0]))
    second["edge_src"][:len(perm)] = second["edge_src"][:len(perm)][perm]
    second["edge_dst"][:len(perm)] = second["edge_dst"][:len(perm)][perm]
    want = [_regular(first), _regular(second)]

    cap_n, cap_e, cap_b = 131072, 524288, 4096
    i32 = dict(dtype=torch.int32, device="cuda")
    bufs = {"op": torch.zeros(cap_n, **i32), "edge_src": torch.zeros(cap_e, **i32),
            "edge_dst": torch.zeros(cap_e, **i32), "node_off": torch.zeros(cap_b + 1, **i32),
            "edge_off": torch.zeros(cap_b + 1, **i32), "seg_id": torch.zeros(cap_n, **i32),
            "graph_env": torch.zeros(cap_b, **i32), "rowptr": torch.zeros(cap_n + 1, **i32),
            "col": torch.zeros(cap_e, **i32), "status": torch.zeros(1, **i32)}
    for batch, ref in zip([first, second], want):
        got, status = _static(batch, bufs)
        assert status == 0
        for k in KEYS:
            assert np.array_equal(got[k], ref[k]), k

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

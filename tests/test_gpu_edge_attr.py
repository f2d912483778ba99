"""Attributes on the edges (Section 3.3.2 as written): contexts created with edge_attributes = 1 take Eq. 6's
edge attributes from an [E x S] array in input edge order, which the library permutes into CSR order."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util

pytestmark = pytest.mark.gpu


def _with_edge_attr(batch, seed, shuffle=True):
    """Shuffle every graph's edge list (so that CSR slots are a non-trivial permutation of the input edges)
    and attach per-edge attributes."""
    rng = np.random.default_rng(seed)
    b = dict(batch)
    b["edge_src"], b["edge_dst"] = batch["edge_src"].copy(), batch["edge_dst"].copy()
    eo = np.concatenate([[0], np.cumsum(b["n_edges"])])
    if shuffle:
        for g in range(b["num_graphs"]):
            perm = rng.permutation(eo[g + 1] - eo[g]) + eo[g]
            b["edge_src"][eo[g]:eo[g + 1]] = batch["edge_src"][perm]
            b["edge_dst"][eo[g]:eo[g + 1]] = batch["edge_dst"][perm]
    bf = batch["model"]["dtype"] == "bf16"
    b["edge_attr"] = dags.tensor_shape_attributes(dags.make_rng(seed), int(eo[-1]), 8, bf)
    b["model"] = dict(batch["model"], edge_attr=True)
    return b


def _dev_batch(batch):
    import torch
    bf = batch["model"]["dtype"] == "bf16"
    dev = {k: batch[k] for k in ("n_nodes", "n_edges", "env_off")}
    for k in ("op", "edge_src", "edge_dst"):
        dev[k] = torch.from_numpy(batch[k]).cuda()
    for k in ("shape", "edge_attr"):
        t = torch.from_numpy(batch[k]).cuda()
        dev[k] = t.to(torch.bfloat16) if bf else t
    return dev


@pytest.mark.parametrize("where", ["host", "device"])
@pytest.mark.parametrize("cfg,kw", [(1, {}), (2, dict(candidates=7)), (3, dict(candidates=15)),
                                    (4, dict(candidates=5)), (6, dict(candidates=4))])
def test_edge_attributes_match_the_oracle(xo, cfg, kw, where):
    import torch
    b = _with_edge_attr(configs.make_batch(cfg, **kw), 100 + cfg)
    m = b["model"]
    blob, _ = gpu_util.default_weights(b, 50 + cfg)
    want = xo.forward(m, blob, b)
    plain = xo.forward(m, blob, {k: v for k, v in b.items() if k != "edge_attr"})
    assert not np.allclose(want["emb"], plain["emb"])            # the attributes matter
    ag = gpu_util.make_agent(b)
    try:
        ag.set_weights(blob)
        mask = torch.from_numpy(b["mask"]).cuda()
        for rep in range(2):
            out = ag.step(b if where == "host" else _dev_batch(b), mask, graph=(rep == 1))
            torch.cuda.synchronize()
            assert ag.device_status() == 0
            gpu_util.assert_close(out["emb"].cpu().numpy(), want["emb"], m["dtype"], "graph_emb")
            gpu_util.assert_close(out["probs"].cpu().numpy(), want["probs"], m["dtype"], "probs")
            gpu_util.assert_close(out["value"].cpu().numpy(), want["value"], m["dtype"], "value")
    finally:
        ag.close()


@pytest.mark.parametrize("cfg,kw", [(2, dict(candidates=5)), (4, dict(candidates=3))])
def test_edges_carrying_their_producers_features_change_nothing(cfg, kw):
    """edge_attr[e] = shape[producer of e]: the same numbers are added in the same (slot) order, so the result
    equals the node-feature context's bit for bit."""
    import torch
    base = configs.make_batch(cfg, **kw)
    b = _with_edge_attr(base, 7)
    no = np.concatenate([[0], np.cumsum(b["n_nodes"])])
    g_of_edge = np.repeat(np.arange(b["num_graphs"]), b["n_edges"])
    b["edge_attr"] = b["shape"][no[g_of_edge] + b["edge_src"]]
    blob, _ = gpu_util.default_weights(b, 3)
    mask = torch.from_numpy(b["mask"]).cuda()
    outs = []
    for model in (b["model"], dict(b["model"], edge_attr=False)):
        bb = dict(b, model=model)
        ag = gpu_util.make_agent(bb)
        try:
            ag.set_weights(blob)
            outs.append(ag.step(bb, mask, graph=False)["emb"].clone())
            torch.cuda.synchronize()
        finally:
            ag.close()
    assert torch.equal(outs[0], outs[1])


def test_large_graph_packed_by_the_global_kernels_and_ranges(xo, monkeypatch):
    """A graph too large for the per-graph packer (global-memory packing kernels write the permutation) and
    a batch packed range by range from page-locked memory."""
    import torch
    import paper_2304_14698_b200 as xrl
    rng = dags.make_rng(9)
    big = dags.random_dag(rng, 17000, 32, 8, False, window=8)
    small = [dags.random_dag(rng, 50, 32, 8, False) for _ in range(3)]
    b = dags.flatten([big] + small, [0, 4], 3)
    b["model"] = dict(configs.MODEL[1], A_max=3)
    b = _with_edge_attr(b, 21)
    blob, _ = gpu_util.default_weights(b, 4)
    want = xo.forward(b["model"], blob, b)
    got = gpu_util.run_gpu(b, blob)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], "fp32", "graph_emb")
    # ranges: page-locked inputs, small threshold
    monkeypatch.setenv("XRL_PIPELINE_MIN_NODES", "3000")
    b2 = _with_edge_attr(configs.make_batch(3, candidates=9), 22)
    blob2, _ = gpu_util.default_weights(b2, 5)
    want2 = xo.forward(b2["model"], blob2, b2)
    ag = gpu_util.make_agent(b2)
    try:
        ag.set_weights(blob2)
        keep = {k: torch.from_numpy(np.ascontiguousarray(b2[k])).pin_memory() for k in ("op", "edge_src", "edge_dst")}
        shp = ag.storage_shape(b2["shape"])
        keep["shape"] = torch.from_numpy(shp.view(np.int16)).pin_memory()
        ag.batch = xrl.xrl_pack_flat(ag.ctx, 0, b2["n_nodes"], b2["n_edges"], keep["op"].numpy(), keep["shape"].numpy(),
                                     keep["edge_src"].numpy(), keep["edge_dst"].numpy(), b2["env_off"], batch=ag.batch)
        xrl.xrl_batch_set_edge_attr(ag.ctx, ag.batch, ag.storage_shape(b2["edge_attr"]))
        out = ag.forward(torch.from_numpy(b2["mask"]).cuda(), graph=False)
        torch.cuda.synchronize()
        assert ag.device_status() == 0
        gpu_util.assert_close(out["emb"].cpu().numpy(), want2["emb"], "bf16", "graph_emb")
    finally:
        ag.close()


def test_order_of_calls_is_enforced():
    import torch
    import paper_2304_14698_b200 as xrl
    b = _with_edge_attr(configs.make_batch(1), 1)
    blob, _ = gpu_util.default_weights(b, 6)
    ag = gpu_util.make_agent(b)
    plain = gpu_util.make_agent(dict(b, model=dict(b["model"], edge_attr=False)))
    try:
        ag.set_weights(blob)
        mask = torch.from_numpy(b["mask"]).cuda()
        ag.batch = xrl.xrl_pack_flat(ag.ctx, 0, b["n_nodes"], b["n_edges"], b["op"], b["shape"], b["edge_src"],
                                     b["edge_dst"], b["env_off"], batch=ag.batch)
        with pytest.raises(xrl.XrlError) as e:
            ag.forward(mask, graph=False)                     # attributes not given yet
        assert e.value.status == 6
        xrl.xrl_batch_set_edge_attr(ag.ctx, ag.batch, b["edge_attr"])
        ag.forward(mask, graph=False)
        with pytest.raises(xrl.XrlError) as e:
            ag.forward(mask, base_id=torch.from_numpy(b["base_id"]).cuda(), graph=False)
        assert e.value.status == 8                            # no delta encoding with attributes on the edges
        ag.batch = xrl.xrl_pack_flat(ag.ctx, 0, b["n_nodes"], b["n_edges"], b["op"], b["shape"], b["edge_src"],
                                     b["edge_dst"], b["env_off"], batch=ag.batch)
        with pytest.raises(xrl.XrlError) as e:
            ag.forward(mask, graph=False)                     # a new packing needs its attributes again
        assert e.value.status == 6
        plain.set_weights(blob)
        plain.pack({k: v for k, v in b.items() if k != "edge_attr"})
        with pytest.raises(xrl.XrlError) as e:
            xrl.xrl_batch_set_edge_attr(plain.ctx, plain.batch, b["edge_attr"])
        assert e.value.status == 6                            # this context takes the producers' features
        torch.cuda.synchronize()
    finally:
        ag.close()
        plain.close()

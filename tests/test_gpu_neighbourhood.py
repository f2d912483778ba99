"""Eq. 7 with a node's consumers among its neighbours (neighbourhood = 1): the attention layers walk a merged
CSR (producers, then consumers) that the packer builds from a second, reversed packing."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("edge_attr", [False, True])
@pytest.mark.parametrize("cfg,kw", [(1, {}), (2, dict(candidates=7)), (3, dict(candidates=15)),
                                    (4, dict(candidates=5)), (6, dict(candidates=4)),
                                    (5, dict(candidates=3, envs=3))])
def test_both_ways_matches_the_oracle(xo, cfg, kw, edge_attr):
    import torch
    b = configs.make_batch(cfg, **kw)
    b["model"] = dict(b["model"], both_ways=True, edge_attr=edge_attr)
    if edge_attr:
        b["edge_attr"] = dags.tensor_shape_attributes(dags.make_rng(cfg), int(b["n_edges"].sum()), 8,
                                                      b["model"]["dtype"] == "bf16")
    m = b["model"]
    blob, _ = gpu_util.default_weights(b, 80 + cfg)
    want = xo.forward(m, blob, b)
    one_way = xo.forward(dict(m, both_ways=False), blob, b)
    assert not np.allclose(want["emb"], one_way["emb"])
    ag = gpu_util.make_agent(b)
    try:
        ag.set_weights(blob)
        mask = torch.from_numpy(b["mask"]).cuda()
        for rep in range(2):
            out = ag.step(b, mask, sample=True, seed=2, step=rep, graph=(rep == 1))
            torch.cuda.synchronize()
            assert ag.device_status() == 0
            gpu_util.assert_close(out["emb"].cpu().numpy(), want["emb"], m["dtype"], "graph_emb")
            gpu_util.assert_close(out["probs"].cpu().numpy(), want["probs"], m["dtype"], "probs")
            gpu_util.assert_close(out["value"].cpu().numpy(), want["value"], m["dtype"], "value")
        import paper_2304_14698_b200 as xrl
        with pytest.raises(xrl.XrlError) as e:
            ag.forward(mask, base_id=torch.from_numpy(b["base_id"]).cuda(), graph=False)
        assert e.value.status == 8
    finally:
        ag.close()


def test_busy_nodes_both_ways(xo):
    """A producer with hundreds of consumers and a consumer with hundreds of producers on the 512-byte-row
    aggregate (rows beyond the gather list), graphs packed by the global-memory kernels included."""
    rng = dags.make_rng(31)
    n = 600
    base = dags.random_dag(rng, n, 32, 8, True, window=10)
    fan_out = dict(base, edge_src=np.concatenate([base["edge_src"], np.zeros(300, np.int32)]).astype(np.int32),
                   edge_dst=np.concatenate([base["edge_dst"], np.arange(200, 500)]).astype(np.int32))
    big = dags.random_dag(rng, 17000, 32, 8, True, window=6)
    b = dags.flatten([fan_out, big, base], [0, 3], 2)
    b["model"] = dict(configs.MODEL[4], A_max=2, L=2, both_ways=True)
    blob, _ = configs.make_weights(b["model"], 8, readout_scale=1.0 / 6000.0)
    got = gpu_util.run_gpu(b, blob)
    want = xo.forward(b["model"], blob, b)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], "bf16", "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], "bf16", "probs")

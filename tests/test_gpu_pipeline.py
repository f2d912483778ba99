"""Large batches packed from page-locked host memory are copied, packed and encoded range by range (ranges of
whole graphs) so that the bus transfer overlaps the encoder.  XRL_PIPELINE_MIN_NODES lowers the size at
which that starts so that small batches exercise it: every output must still match the oracle."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util

pytestmark = pytest.mark.gpu

KEYS = ("node_off", "edge_off", "seg_id", "graph_env", "rowptr", "col")


def _pinned(ag, batch):
    import torch
    keep = {k: torch.from_numpy(np.ascontiguousarray(batch[k])).pin_memory() for k in ("op", "edge_src", "edge_dst")}
    shp = ag.storage_shape(batch["shape"])
    keep["shape"] = torch.from_numpy(shp.view(np.int16) if shp.dtype == np.uint16 else shp).pin_memory()
    return keep


def _pack_pinned(xrl, ag, batch, keep):
    ag.batch = xrl.xrl_pack_flat(ag.ctx, 0, batch["n_nodes"], batch["n_edges"], keep["op"].numpy(),
                                 keep["shape"].numpy(), keep["edge_src"].numpy(), keep["edge_dst"].numpy(),
                                 batch["env_off"], batch=ag.batch)


@pytest.mark.parametrize("cfg,kw,min_nodes", [(3, dict(candidates=15), 2000), (4, dict(candidates=9), 9000),
                                              (5, dict(candidates=7, envs=3), 5000), (2, dict(candidates=11), 3500),
                                              (1, {}, 100)])
def test_ranges_of_graphs_match_the_oracle(xo, monkeypatch, cfg, kw, min_nodes):
    import torch
    import paper_2304_14698_b200 as xrl
    monkeypatch.setenv("XRL_PIPELINE_MIN_NODES", str(min_nodes))
    batch = configs.make_batch(cfg, **kw)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 70 + cfg)
    st, want_pack = xo.pack(batch)
    assert st == 0
    want = xo.forward(m, blob, batch)
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        keep = _pinned(ag, batch)
        mask = torch.from_numpy(batch["mask"]).cuda()
        for rep in range(2):                       # the second pack re-uses the batch, its stream and events
            _pack_pinned(xrl, ag, batch, keep)
            ranged_launches = xrl.xrl_launch_counts(ag.ctx)["pack"]
            out = ag.forward(mask, sample=True, seed=5, step=rep, graph=False)
            torch.cuda.synchronize()
            assert ag.device_status() == 0
            got_pack = xrl.xrl_batch_export(ag.batch)
            for k in KEYS:
                assert np.array_equal(got_pack[k], want_pack[k]), k
            dt = m["dtype"]
            gpu_util.assert_close(out["emb"].cpu().numpy(), want["emb"], dt, "graph_emb")
            gpu_util.assert_close(out["probs"].cpu().numpy(), want["probs"], dt, "probs")
            gpu_util.assert_close(out["value"].cpu().numpy(), want["value"], dt, "value")
            assert np.array_equal(out["action"].cpu().numpy(), xo.sample(out["probs"].cpu().numpy(), 5, rep))
        # the same batch object packed in one piece again (device inputs), then delta encoding on ranges
        monkeypatch.delenv("XRL_PIPELINE_MIN_NODES")
        out1 = {k: v.clone() for k, v in ag.step(batch, mask, graph=False).items()}
        assert xrl.xrl_launch_counts(ag.ctx)["pack"] < ranged_launches      # one packing launch instead of one per range
        monkeypatch.setenv("XRL_PIPELINE_MIN_NODES", str(min_nodes))
        _pack_pinned(xrl, ag, batch, keep)
        if cfg != 1:
            base = torch.from_numpy(batch["base_id"]).cuda()
            out2 = ag.forward(mask, base_id=base, graph=False)
            torch.cuda.synchronize()
            gpu_util.assert_close(out2["emb"].cpu().numpy(), want["emb"], m["dtype"], "graph_emb (delta)")
        gpu_util.assert_close(out1["emb"].cpu().numpy(), want["emb"], m["dtype"], "graph_emb (one piece)")
    finally:
        ag.close()


def test_bad_graph_in_a_late_range_is_reported(monkeypatch):
    import torch
    import paper_2304_14698_b200 as xrl
    monkeypatch.setenv("XRL_PIPELINE_MIN_NODES", "100")
    batch = configs.make_batch(1)
    batch["edge_src"] = batch["edge_src"].copy()
    batch["edge_src"][-1] = 10 ** 6              # an endpoint outside the last graph
    ag = gpu_util.make_agent(batch)
    try:
        keep = _pinned(ag, batch)
        _pack_pinned(xrl, ag, batch, keep)
        assert ag.device_status() == 2            # XRL_ERR_BAD_GRAPH, without any encode call in between
    finally:
        ag.close()

"""One submission per step (xrl_graph_begin / xrl_graph_launch): the recorded kernels must give exactly
what the direct launches give, across steps of different sizes that reuse one executable graph."""
import numpy as np
import pytest

from workloads import configs
import gpu_util

pytestmark = pytest.mark.gpu


def _dev_batch(batch):
    import torch
    dev = {k: batch[k] for k in ("n_nodes", "n_edges", "env_off")}
    dev["op"] = torch.from_numpy(batch["op"]).cuda()
    shp = torch.from_numpy(batch["shape"]).cuda()
    dev["shape"] = shp.to(torch.bfloat16) if batch["model"]["dtype"] == "bf16" else shp
    dev["edge_src"] = torch.from_numpy(batch["edge_src"]).cuda()
    dev["edge_dst"] = torch.from_numpy(batch["edge_dst"]).cuda()
    return dev


@pytest.mark.parametrize("cfg", [1, 2, 6])
def test_recorded_steps_equal_direct_launches(xo, cfg):
    import torch
    big = configs.make_batch(cfg)
    blob, _ = gpu_util.default_weights(big, 40 + cfg)
    ag = gpu_util.make_agent(big)
    try:
        ag.set_weights(blob)
        sizes = [None, 3, 1, 5, None, 0] if cfg != 1 else [None, 2, 7, 0, None]
        for i, c in enumerate(sizes):
            b = big if c is None else configs.make_batch(cfg, candidates=c)
            dev = _dev_batch(b)
            mask = torch.from_numpy(b["mask"]).cuda()
            direct = {k: v.clone() for k, v in ag.step(dev, mask, sample=True, seed=3, step=i, graph=False).items()}
            rec = ag.step(dev, mask, sample=True, seed=3, step=i, graph=True)
            torch.cuda.synchronize()
            assert ag.device_status() == 0
            for k in ("emb", "probs", "value", "action"):
                assert torch.equal(direct[k], rec[k]), (cfg, i, k)
        # the last recorded step against the oracle
        want = xo.forward(b["model"], blob, b)
        dt = b["model"]["dtype"]
        gpu_util.assert_close(rec["emb"].cpu().numpy(), want["emb"], dt, "graph_emb")
        gpu_util.assert_close(rec["probs"].cpu().numpy(), want["probs"], dt, "probs")
    finally:
        ag.close()


def test_what_cannot_be_recorded_is_refused():
    import torch
    import paper_2304_14698_b200 as xrl
    batch = configs.make_batch(1)
    blob, _ = gpu_util.default_weights(batch, 2)
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        dev = _dev_batch(batch)
        mask = torch.from_numpy(batch["mask"]).cuda()
        ag.step(dev, mask, graph=False)
        with pytest.raises(xrl.XrlError) as e:
            xrl.xrl_graph_launch(ag.ctx)                 # nothing is being recorded
        assert e.value.status == 6
        xrl.xrl_graph_begin(ag.ctx)
        for call in (lambda: xrl.xrl_graph_begin(ag.ctx), lambda: ag.pack(dev), lambda: xrl.xrl_profile(ag.ctx, True),
                     lambda: ag.device_status()):
            with pytest.raises(xrl.XrlError) as e:
                call()
            assert e.value.status == 6
        xrl.xrl_graph_launch(ag.ctx)                     # an empty recording is a valid (empty) graph
        xrl.xrl_profile(ag.ctx, True)
        with pytest.raises(xrl.XrlError) as e:
            xrl.xrl_graph_begin(ag.ctx)                  # event timing needs direct launches
        assert e.value.status == 6
        out = ag.step(dev, mask, graph=True)             # the agent falls back to direct launches
        xrl.xrl_profile(ag.ctx, False)
        torch.cuda.synchronize()
        assert ag.device_status() == 0 and bool(torch.isfinite(out["probs"]).all())
    finally:
        ag.close()

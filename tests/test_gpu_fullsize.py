"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (device-resident
inputs, Agent.step).  For the two largest workloads (the 1,024-action step and the 64-environment
rollout batch) the oracle runs the whole batch once per module; the packed arrays are then compared bit
for bit and every graph embedding, every probability of every environment and slot, and every value
estimate element by element within the bf16 tolerance, for the full encoder and for the delta encoder.
The draw is exact given the probabilities the GPU reports."""
import numpy as np
import pytest

from workloads import configs
import gpu_util

pytestmark = pytest.mark.gpu

_cache = {}


def _reference(xo, cfg_id):
    """The oracle's whole step on workload `cfg_id` at full size (computed once, kept for the module)."""
    if cfg_id not in _cache:
        batch = configs.make_batch(cfg_id)
        blob, _ = gpu_util.default_weights(batch, 1000 + cfg_id)
        _cache[cfg_id] = (batch, blob, xo.forward(batch["model"], blob, batch))
    return _cache[cfg_id]


def _run_full(batch, blob, seed, step, delta=False):
    import torch
    import paper_2304_14698_b200 as xrl
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        dev = {k: batch[k] for k in ("n_nodes", "n_edges", "env_off")}
        dev["op"] = torch.from_numpy(batch["op"]).cuda()
        shp = torch.from_numpy(batch["shape"]).cuda()
        dev["shape"] = shp.to(torch.bfloat16) if batch["model"]["dtype"] == "bf16" else shp
        dev["edge_src"] = torch.from_numpy(batch["edge_src"]).cuda()
        dev["edge_dst"] = torch.from_numpy(batch["edge_dst"]).cuda()
        mask = torch.from_numpy(batch["mask"]).cuda()
        bid = torch.from_numpy(batch["base_id"]).cuda() if delta else None
        out = ag.step(dev, mask, sample=True, seed=seed, step=step, base_id=bid)
        torch.cuda.synchronize()
        res = {k: v.cpu().numpy() for k, v in out.items()}
        res["status"] = ag.device_status()
        res["packed"] = xrl.xrl_batch_export(ag.batch)
        return res
    finally:
        ag.close()


def _check(xo, cfg_id, delta=False):
    batch, blob, want = _reference(xo, cfg_id)
    m = batch["model"]
    got = _run_full(batch, blob, seed=cfg_id, step=3, delta=delta)
    assert got["status"] == 0

    for k in ("node_off", "edge_off", "seg_id", "graph_env", "rowptr", "col"):
        assert np.array_equal(got["packed"][k], want["packed"][k]), k

    what = f"workload {cfg_id}{' (delta)' if delta else ''} "
    gpu_util.assert_close(got["emb"], want["emb"], m["dtype"], what + "graph_emb, every graph")
    gpu_util.assert_close(got["probs"], want["probs"], m["dtype"], what + "probs, every environment and slot")
    gpu_util.assert_close(got["value"], want["value"], m["dtype"], what + "value, every environment")

    probs = got["probs"]
    A = m["A_max"]
    n_env = len(batch["env_off"]) - 1
    full_mask = np.concatenate([batch["mask"], np.ones((n_env, 1), np.uint8)], axis=1)
    assert np.all(probs[full_mask == 0] == 0.0)
    assert np.all(probs[full_mask == 1] >= 0.0)
    assert np.all(np.abs(probs.sum(axis=1) - 1.0) < 1e-4)
    assert np.all(probs[:, A] > 0)
    # the draw is exact given the probabilities the GPU reports
    assert np.array_equal(got["action"], xo.sample(probs, cfg_id, 3))


def test_large_step_full_size_every_output(xo):
    _check(xo, 4)


def test_large_step_full_size_delta_encoding_every_output(xo):
    _check(xo, 4, delta=True)


def test_rollout_batch_full_size_every_output(xo):
    _check(xo, 5)


def test_rollout_batch_full_size_delta_encoding_every_output(xo):
    _check(xo, 5, delta=True)


def test_cnn_step_full_size_every_output(xo):
    batch = configs.make_batch(3)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 1003)
    got = gpu_util.run_gpu(batch, blob, where="device")
    want = xo.forward(m, blob, batch)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], "bf16", "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], "bf16", "probs")
    gpu_util.assert_close(got["value"], want["value"], "bf16", "value")

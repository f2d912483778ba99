"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (device-resident
inputs, Agent.step).  The packed arrays are compared bit for bit in full; graph embeddings are
compared on sampled graphs the oracle encodes one by one; the policy is checked through its
structural properties and through log-probability differences of the sampled graphs."""
import numpy as np
import pytest

from workloads import configs
import gpu_util

pytestmark = pytest.mark.gpu


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


def _check(xo, cfg_id, n_sample, delta=False):
    batch = configs.make_batch(cfg_id)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 1000 + cfg_id)
    got = _run_full(batch, blob, seed=cfg_id, step=3, delta=delta)
    assert got["status"] == 0

    st, packed = xo.pack(batch)
    assert st == 0
    for k in ("node_off", "edge_off", "seg_id", "graph_env", "rowptr", "col"):
        assert np.array_equal(got["packed"][k], packed[k]), k

    rng = np.random.default_rng(cfg_id)
    env_off = batch["env_off"]
    e = int(rng.integers(0, len(env_off) - 1))
    cur = int(env_off[e])
    C = int(env_off[e + 1]) - cur - 1
    valid = np.flatnonzero(batch["mask"][e, :C])
    picks = rng.choice(valid, size=min(n_sample - 1, len(valid)), replace=False)
    sel = np.array([cur] + [cur + 1 + int(a) for a in picks], dtype=np.int32)
    want = xo.encode(m, blob, batch, packed, sel=sel)["emb"]
    gpu_util.assert_close(got["emb"][sel], want, m["dtype"], f"cfg{cfg_id} sampled graph_emb")

    probs = got["probs"]
    A = m["A_max"]
    full_mask = np.concatenate([batch["mask"], np.ones((len(env_off) - 1, 1), np.uint8)], axis=1)
    assert np.all(probs[full_mask == 0] == 0.0)
    assert np.all(probs[full_mask == 1] >= 0.0)
    assert np.all(np.abs(probs.sum(axis=1) - 1.0) < 1e-4)
    assert np.all(probs[:, A] > 0)
    assert np.all(np.isfinite(got["value"]))
    # log-probability differences against the oracle's logits of the sampled graphs
    mini = {"env_off": np.array([0, len(sel)], np.int32), "mask": np.ones((1, len(sel) - 1), np.uint8)}
    st, logits, _, _ = xo.policy_value(dict(m, A_max=len(sel) - 1), blob, mini, want)
    assert st == 0
    for i, a in enumerate(picks):
        lhs = np.log(probs[e, a]) - np.log(probs[e, A])
        rhs = logits[0, i] - logits[0, -1]
        assert abs(lhs - rhs) < 5e-2, (a, lhs, rhs)
    # the draw is exact given the probabilities the GPU reports
    assert np.array_equal(got["action"], xo.sample(probs, cfg_id, 3))


def test_large_step_full_size(xo):
    _check(xo, 4, 6)


def test_rollout_batch_full_size(xo):
    _check(xo, 5, 6)


def test_large_step_full_size_delta_encoding(xo):
    _check(xo, 4, 6, delta=True)


def test_rollout_batch_full_size_delta_encoding(xo):
    _check(xo, 5, 6, delta=True)


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

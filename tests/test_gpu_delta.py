"""Delta encoding (xrl_encode_delta) against the same oracle as the full encoder: the oracle encodes
every candidate in full; the library recomputes only the rows a rewrite can reach."""
import numpy as np
import pytest

from workloads import configs
import gpu_util

pytestmark = pytest.mark.gpu


def _run_delta(batch, blob, base_id):
    import torch
    import paper_2304_14698_b200 as xrl
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        ag.pack(batch)
        bid = None if base_id is None else torch.from_numpy(np.ascontiguousarray(base_id, dtype=np.int32)).cuda()
        mask = torch.from_numpy(batch["mask"]).cuda()
        o = ag.forward(mask, base_id=bid) if bid is not None else None
        if bid is None:
            emb = torch.empty((batch["num_graphs"], batch["model"]["H"]), device="cuda")
            xrl.xrl_encode_delta(ag.ctx, ag.batch, None, emb)
            o = {"emb": emb}
        torch.cuda.synchronize()
        res = {k: v.cpu().numpy() for k, v in o.items()}
        res["status"] = ag.device_status()
        res["rows"] = xrl.xrl_delta_rows(ag.ctx, batch["model"]["L"])
        return res
    finally:
        ag.close()


@pytest.mark.parametrize("cfg,kw", [(2, {}), (3, dict(candidates=31)), (4, dict(candidates=15)),
                                    (5, dict(candidates=7, envs=4))])
def test_delta_matches_oracle(xo, cfg, kw):
    batch = configs.make_batch(cfg, **kw)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 1000 + cfg)
    got = _run_delta(batch, blob, batch["base_id"])
    assert got["status"] == 0
    want = xo.forward(m, blob, batch)
    gpu_util.assert_close(got["emb"], want["emb"], m["dtype"], "graph_emb (delta)")
    gpu_util.assert_close(got["probs"], want["probs"], m["dtype"], "probs (delta)")
    gpu_util.assert_close(got["value"], want["value"], m["dtype"], "value (delta)")
    N = int(batch["n_nodes"].sum())
    rows = got["rows"]
    assert all(rows[i] <= rows[i + 1] for i in range(len(rows) - 1))     # the change only spreads
    assert rows[-1] < N // 2                                             # and stays local


def test_delta_equals_full_encode_bit_for_bit_without_hints(xo):
    """No hint: every row is recomputed, in the same kernels, so the result is the full encoder's."""
    batch = configs.make_batch(3, candidates=7)
    blob, _ = gpu_util.default_weights(batch, 5)
    full = gpu_util.run_gpu(batch, blob)
    got = _run_delta(batch, blob, None)
    assert got["rows"][0] == int(batch["n_nodes"].sum())
    np.testing.assert_allclose(got["emb"], full["emb"], rtol=1e-5, atol=1e-6)


def test_wrong_hints_cost_time_not_correctness(xo):
    batch = configs.make_batch(2, candidates=15)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 6)
    rng = np.random.default_rng(0)
    bad = batch["base_id"].copy()
    idx = rng.choice(len(bad), size=len(bad) // 3, replace=False)
    bad[idx] = rng.integers(-5, len(bad) + 5, size=len(idx))             # random, out-of-range, wrong graph ...
    good = _run_delta(batch, blob, batch["base_id"])
    got = _run_delta(batch, blob, bad)
    want = xo.forward(m, blob, batch)
    gpu_util.assert_close(got["emb"], want["emb"], m["dtype"], "graph_emb (bad hints)")
    assert got["rows"][0] > good["rows"][0]


def test_delta_with_independent_graphs_and_no_layers(xo):
    batch = configs.make_batch(1)                # candidates are unrelated DAGs: nothing to reuse
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 7)
    got = _run_delta(batch, blob, batch["base_id"])
    want = xo.forward(m, blob, batch)
    gpu_util.assert_close(got["emb"], want["emb"], "fp32", "graph_emb")
    batch0 = configs.make_batch(2, candidates=5)
    batch0["model"] = dict(batch0["model"], L=0)
    blob0, _ = gpu_util.default_weights(batch0, 8)
    got0 = _run_delta(batch0, blob0, batch0["base_id"])
    want0 = xo.forward(batch0["model"], blob0, batch0)
    gpu_util.assert_close(got0["emb"], want0["emb"], "fp32", "graph_emb L=0")

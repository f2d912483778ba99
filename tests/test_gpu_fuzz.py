"""Randomised parity: many small batches with random graph shapes, model sizes, masks and hints,
each compared with the oracle (pack bit for bit, floats within tolerance, full and delta encoding)."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util

pytestmark = pytest.mark.gpu

SHAPES = [(32, 1), (32, 4), (64, 2), (64, 8), (96, 3), (128, 4), (128, 16), (256, 8), (256, 4)]


def _random_case(seed):
    rng = np.random.default_rng(seed)
    H, K = SHAPES[rng.integers(len(SHAPES))]
    dtype = "bf16" if rng.random() < 0.5 else "fp32"
    T = int(rng.choice([3, 17, 32, 64]))
    m = dict(T=T, S=8, H=H, K=K, L=int(rng.integers(0, 4)), Hm=int(rng.integers(1, 70)),
             Hm2=int(rng.integers(1, 50)) if rng.random() < 0.4 else 0,
             Dg=int(rng.integers(0, 4)), dtype=dtype, A_max=0)
    nenv = int(rng.integers(1, 4))
    graphs, env_off = [], [0]
    grng = dags.make_rng(seed + 1000)
    for _ in range(nenv):
        n = int(rng.integers(1, 200))
        cur = dags.random_dag(grng, n, T, 8, dtype == "bf16", window=int(rng.integers(1, 20)))
        if n > 3 and rng.random() < 0.5:          # repeated edges and one busy consumer
            extra = int(rng.integers(1, 60))
            cur["edge_src"] = np.concatenate([cur["edge_src"], rng.integers(0, n - 1, extra)]).astype(np.int32)
            cur["edge_dst"] = np.concatenate([cur["edge_dst"], np.full(extra, n - 1)]).astype(np.int32)
        graphs.append(cur)
        for _c in range(int(rng.integers(0, 6))):
            if n > 12 and rng.random() < 0.7:
                graphs.append(dags.local_rewrite(grng, cur, T, dtype == "bf16"))
            elif rng.random() < 0.1:
                graphs.append({"op": np.zeros(0, np.int32), "shape": np.zeros((0, 8), np.float32),
                               "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)})
            else:
                graphs.append(dags.random_dag(grng, int(rng.integers(1, 150)), T, 8, dtype == "bf16"))
        env_off.append(len(graphs))
    A = max(env_off[e + 1] - env_off[e] - 1 for e in range(nenv)) + int(rng.integers(0, 3))
    m["A_max"] = A
    batch = dags.flatten(graphs, env_off, A)
    batch["mask"][rng.random(batch["mask"].shape) < 0.2] = 0
    # every third case or so: attributes on the edges and / or neighbourhoods read both ways
    if rng.random() < 0.35:
        m["edge_attr"] = True
        batch["edge_attr"] = dags.tensor_shape_attributes(grng, int(batch["n_edges"].sum()), 8, dtype == "bf16")
    if rng.random() < 0.35:
        m["both_ways"] = True
    batch["model"] = m
    # spoil some hints
    hint = batch["base_id"].copy()
    spoil = rng.random(len(hint)) < 0.05
    hint[spoil] = rng.integers(-3, len(hint) + 3, size=int(spoil.sum()))
    blob, _ = configs.make_weights(m, seed, readout_scale=1.0 / max(1.0, float(batch["n_nodes"].mean())))
    g0 = rng.normal(size=(len(graphs), m["Dg"])) if m["Dg"] and rng.random() < 0.5 else None
    return batch, m, blob, hint, g0


@pytest.mark.parametrize("seed", range(32))
def test_random_batches(xo, seed):
    import torch
    import paper_2304_14698_b200 as xrl
    batch, m, blob, hint, g0 = _random_case(seed)
    st, packed = xo.pack(batch)
    assert st == 0
    enc = xo.encode(m, blob, batch, packed, g0=g0)
    st, _, probs, value = xo.policy_value(m, blob, batch, enc["emb"])
    assert st == 0
    ag = gpu_util.make_agent(batch, slack=3)
    try:
        ag.set_weights(blob)
        ag.pack(batch)
        got_pack = xrl.xrl_batch_export(ag.batch)
        for k in ("node_off", "edge_off", "seg_id", "graph_env", "rowptr", "col"):
            assert np.array_equal(got_pack[k], packed[k]), (seed, k)
        g0d = None if g0 is None else torch.from_numpy(g0.astype(np.float32)).cuda()
        mask = torch.from_numpy(batch["mask"]).cuda()
        # delta encoding is defined for the default reading only (producers' features, producers as neighbours)
        for mode in ("full",) if (m.get("edge_attr") or m.get("both_ways")) else ("full", "delta"):
            bid = torch.from_numpy(hint).cuda() if mode == "delta" else None
            o = ag.forward(mask, sample=True, seed=seed, step=7, g0=g0d, base_id=bid)
            torch.cuda.synchronize()
            assert ag.device_status() == 0
            gpu_util.assert_close(o["emb"].cpu().numpy(), enc["emb"], m["dtype"], f"seed {seed} {mode} emb")
            gpu_util.assert_close(o["probs"].cpu().numpy(), probs, m["dtype"], f"seed {seed} {mode} probs")
            gpu_util.assert_close(o["value"].cpu().numpy(), value, m["dtype"], f"seed {seed} {mode} value")
            p = o["probs"].cpu().numpy()
            assert np.all(p[probs == 0] == 0.0)
            assert np.array_equal(o["action"].cpu().numpy(), xo.sample(p, seed, 7))
    finally:
        ag.close()

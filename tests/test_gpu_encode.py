"""GPU parity of the encoder and heads (Sections 3.3.2-3.4) against the CPU oracle."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util

pytestmark = pytest.mark.gpu

CASES = [(1, {}), (2, {}), (3, dict(candidates=15)), (4, dict(candidates=7)),
         (5, dict(candidates=7, envs=3)), (6, {})]     # 6: the paper's hyper-parameter table (k = 5, heads [256, 64])


def _oracle(xo, batch, blob, **kw):
    st, packed = xo.pack(batch)
    assert st == 0
    return packed, xo.encode(batch["model"], blob, batch, packed, **kw)


@pytest.mark.parametrize("cfg,kw", CASES)
def test_node_features_after_each_stage(xo, cfg, kw):
    """Eq. 6 and each attention layer, node by node."""
    import paper_2304_14698_b200 as xrl
    batch = configs.make_batch(cfg, **kw)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 1000 + cfg)
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        ag.pack(batch)
        for layer in range(m["L"] + 1):
            got = xrl.xrl_debug_node_features(ag.ctx, ag.batch, layer, m["H"])
            _, want = _oracle(xo, batch, blob, dump_layer=layer, want_nodes=True)
            gpu_util.assert_close(got, want["nodes"], m["dtype"], f"cfg{cfg} nodes after stage {layer}")
        assert ag.device_status() == 0
    finally:
        ag.close()


@pytest.mark.parametrize("where", ["host", "device"])
@pytest.mark.parametrize("cfg,kw", CASES)
def test_step_outputs(xo, cfg, kw, where):
    """graph_emb, probs, value of the whole step; structural properties of probs."""
    batch = configs.make_batch(cfg, **kw)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 1000 + cfg)
    got = gpu_util.run_gpu(batch, blob, where=where)
    assert got["status"] == 0
    want = xo.forward(m, blob, batch)
    gpu_util.assert_close(got["emb"], want["emb"], m["dtype"], "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], m["dtype"], "probs")
    gpu_util.assert_close(got["value"], want["value"], m["dtype"], "value")
    assert np.all(got["probs"][want["probs"] == 0] == 0.0)       # masked / padded: exactly zero
    assert np.all(np.abs(got["probs"].sum(axis=1) - 1) < 1e-5)
    assert np.all(got["probs"][:, -1] > 0)


def test_policy_with_spread_logits(xo):
    """Head weights scaled so that the candidates get clearly different probabilities."""
    batch = configs.make_batch(2, candidates=31)
    m = batch["model"]
    blob, W = gpu_util.default_weights(batch, 77)
    W["pw2"] *= 400.0
    blob = configs.pack_weights(m, W)
    got = gpu_util.run_gpu(batch, blob)
    want = xo.forward(m, blob, batch)
    assert want["probs"][0, :31].max() / want["probs"][0, :31].min() > 1.5
    gpu_util.assert_close(got["probs"], want["probs"], "fp32", "probs")


def test_global_attribute_input(xo):
    import torch
    import paper_2304_14698_b200 as xrl
    batch = configs.make_batch(1)
    m = dict(batch["model"], Dg=3)
    batch["model"] = m
    blob, _ = gpu_util.default_weights(batch, 5)
    g0 = np.random.default_rng(0).normal(size=(8, 3))
    _, want = _oracle(xo, batch, blob, g0=g0)
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        ag.pack(batch)
        emb = torch.empty((8, m["H"]), device="cuda")
        xrl.xrl_encode(ag.ctx, ag.batch, emb, torch.from_numpy(g0.astype(np.float32)).cuda())
        gpu_util.assert_close(emb.cpu().numpy(), want["emb"], "fp32", "emb with g0")
    finally:
        ag.close()


@pytest.mark.parametrize("Hm,Hm2", [(256, 64), (64, 256), (1, 1), (1024, 1024), (33, 7)])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_heads_with_two_hidden_layers(xo, Hm, Hm2, dtype):
    """Policy and value MLPs with a second hidden layer: widths below, at and above the thread-block
    size, several environments, masked candidates, sampling."""
    batch = configs.make_batch(5, candidates=5, envs=3, nodes_scale=0.2)
    batch["mask"][1, 2] = 0
    m = dict(batch["model"], H=64, K=2, L=1, Hm=Hm, Hm2=Hm2, dtype=dtype)
    batch["model"] = m
    blob, _ = gpu_util.default_weights(batch, 31)
    got = gpu_util.run_gpu(batch, blob, sample=True, seed=9, step=4)
    want = xo.forward(m, blob, batch)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], dtype, "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], dtype, "probs")
    gpu_util.assert_close(got["value"], want["value"], dtype, "value")
    assert np.array_equal(got["action"], xo.sample(got["probs"], 9, 4))


@pytest.mark.parametrize("H,K,dtype,L", [(32, 1, "fp32", 1), (32, 4, "bf16", 1), (96, 3, "fp32", 2),
                                          (96, 2, "bf16", 2), (256, 8, "fp32", 1), (512, 8, "fp32", 1),
                                          (512, 16, "bf16", 1), (64, 8, "bf16", 0), (128, 2, "bf16", 2)])
def test_model_shapes(xo, H, K, dtype, L):
    """Every row geometry of the row-wise kernels (lanes per row, vectors per lane), L = 0."""
    batch = configs.make_batch(1)
    if dtype == "bf16":
        batch["shape"] = dags.round_to_bf16_grid(batch["shape"])
    m = dict(batch["model"], H=H, K=K, dtype=dtype, L=L, Hm=40)
    batch["model"] = m
    blob, _ = gpu_util.default_weights(batch, 9)
    got = gpu_util.run_gpu(batch, blob)
    want = xo.forward(m, blob, batch)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], dtype, "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], dtype, "probs")
    gpu_util.assert_close(got["value"], want["value"], dtype, "value")


@pytest.mark.parametrize("H,K,dtype", [(96, 3, "bf16"), (160, 5, "fp32"), (64, 2, "fp32")])
def test_cuda_core_transform_on_many_rows(xo, H, K, dtype):
    """Row counts large enough for the 128 x 128 tile of the CUDA-core transform, sizes the tensor-core
    kernel does not take."""
    batch = configs.make_batch(2, candidates=19)
    if dtype == "bf16":
        batch["shape"] = dags.round_to_bf16_grid(batch["shape"])
    m = dict(batch["model"], H=H, K=K, dtype=dtype, L=2, Hm=32)
    batch["model"] = m
    blob, _ = gpu_util.default_weights(batch, 12)
    got = gpu_util.run_gpu(batch, blob)
    want = xo.forward(m, blob, batch)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], dtype, "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], dtype, "probs")


def test_cuda_core_kernels_on_tensor_core_shapes(xo, monkeypatch):
    """XRL_FORCE_SIMT_TRANSFORM keeps Eq. 6 and the transform on the CUDA cores for shapes the tensor-core
    kernels normally take: both paths must agree with the oracle."""
    monkeypatch.setenv("XRL_FORCE_SIMT_TRANSFORM", "1")
    batch = configs.make_batch(4, candidates=3)
    blob, _ = gpu_util.default_weights(batch, 1004)
    got = gpu_util.run_gpu(batch, blob)
    want = xo.forward(batch["model"], blob, batch)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], "bf16", "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], "bf16", "probs")


@pytest.mark.parametrize("cfg,kw", [(4, dict(candidates=3)), (2, dict(candidates=7)), (3, dict(candidates=7))])
def test_large_attention_scores(xo, cfg, kw):
    """Attention vectors scaled up until the scores of one row differ by hundreds: the running softmax
    has to move its reference exponent (a rarely taken branch) and must neither overflow nor lose the
    dominant producer."""
    batch = configs.make_batch(cfg, **kw)
    m = batch["model"]
    _, W = gpu_util.default_weights(batch, 31)
    for l in range(1, m["L"] + 1):
        W[f"a_src{l}"] *= 300.0
        W[f"a_dst{l}"] *= 300.0
    blob = configs.pack_weights(m, W)
    got = gpu_util.run_gpu(batch, blob)
    st, packed = xo.pack(batch)
    enc = xo.encode(m, blob, batch, packed, dump_layer=1, want_nodes=True, want_alpha=True)
    assert np.nanmax(enc["alpha_edge"]) > 0.999 and np.nanmin(enc["alpha_edge"]) < 1e-30   # really saturated
    assert got["status"] == 0
    assert np.all(np.isfinite(got["emb"]))
    if m["dtype"] == "fp32":
        gpu_util.assert_close(got["emb"], enc["emb"], "fp32", "graph_emb")
    else:
        # with saturated attention a bf16 rounding of Z can flip which producer wins: compare the bulk
        err = np.abs(got["emb"] - enc["emb"])
        bound = 2e-2 + 2e-2 * np.abs(enc["emb"])
        assert (err <= bound).mean() > 0.97


@pytest.mark.parametrize("cfg", [2, 4])
def test_one_context_many_batches(xo, cfg):
    """A context and its batch object are reused for steps of different sizes (the candidate set shrinks and
    grows between rewrite steps): nothing may leak from one step into the next, in either encoder."""
    import torch
    big = configs.make_batch(cfg, candidates=9, seed=50)
    m = big["model"]
    blob, _ = gpu_util.default_weights(big, 77)
    ag = gpu_util.make_agent(big, slack=64)
    try:
        ag.set_weights(blob)
        for step, cands in enumerate([9, 2, 7, 0, 5]):
            batch = configs.make_batch(cfg, candidates=cands, seed=60 + step)
            want = xo.forward(m, blob, batch)
            mask = torch.from_numpy(batch["mask"]).cuda()
            for mode in ("full", "delta"):
                bid = torch.from_numpy(batch["base_id"]).cuda() if mode == "delta" else None
                o = ag.step(batch, mask, sample=True, seed=1, step=step, base_id=bid)
                torch.cuda.synchronize()
                assert ag.device_status() == 0
                gpu_util.assert_close(o["emb"].cpu().numpy(), want["emb"], m["dtype"], f"step {step} {mode} emb")
                gpu_util.assert_close(o["probs"].cpu().numpy(), want["probs"], m["dtype"], f"step {step} {mode} probs")
                gpu_util.assert_close(o["value"].cpu().numpy(), want["value"], m["dtype"], f"step {step} {mode} value")
    finally:
        ag.close()


def test_degenerate_batches(xo):
    """Environment without candidates, fully masked environment, empty graph, isolated nodes,
    a consumer with hundreds of producers, padded action slots."""
    rng = dags.make_rng(11)
    n = 400
    star = {"op": rng.integers(0, 32, n).astype(np.int32), "shape": dags.shape_features(rng, n, 8, False),
            "edge_src": np.arange(n - 1, dtype=np.int32), "edge_dst": np.full(n - 1, n - 1, np.int32)}
    iso = {"op": rng.integers(0, 32, 7).astype(np.int32), "shape": dags.shape_features(rng, 7, 8, False),
           "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)}
    empty = {"op": np.zeros(0, np.int32), "shape": np.zeros((0, 8), np.float32),
             "edge_src": np.zeros(0, np.int32), "edge_dst": np.zeros(0, np.int32)}
    g = [dags.random_dag(rng, 30) for _ in range(4)]
    graphs = [g[0],                 # env 0: no candidates
              g[1], star, iso,      # env 1: two candidates, both masked below
              g[2], empty, g[3], star]   # env 2
    b = dags.flatten(graphs, [0, 1, 4, 8], 5)
    b["mask"][1, :] = 0
    b["model"] = dict(configs.MODEL[1], A_max=5)
    blob, _ = configs.make_weights(b["model"], 3, readout_scale=0.02)
    got = gpu_util.run_gpu(b, blob)
    want = xo.forward(b["model"], blob, b)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], "fp32", "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], "fp32", "probs")
    gpu_util.assert_close(got["value"], want["value"], "fp32", "value")
    assert got["probs"][0, -1] == 1.0 and got["probs"][1, -1] == 1.0
    assert np.all(got["probs"][want["probs"] == 0] == 0.0)


@pytest.mark.parametrize("H,K,dtype", [(256, 8, "bf16"), (256, 4, "bf16"), (256, 16, "bf16"), (128, 4, "fp32")])
def test_busy_consumers_on_512_byte_rows(xo, H, K, dtype):
    """Consumers with more producers than the gather list of the 512-byte-row aggregate holds (160 entries
    per 32 rows), alone and next to ordinary rows, on every row geometry that kernel takes; with the last
    attention layer fused with the per-graph sum (L = 2) and without it (intermediate layer)."""
    rng = dags.make_rng(23)
    bf = dtype == "bf16"
    n = 700
    # node n - 1 has 400 producers, node n - 2 has 170, node 300 has 161 (with repeats), the rest few
    src = [np.arange(0, 400), np.arange(100, 270), rng.integers(0, 299, 161)]
    dst = [np.full(400, n - 1), np.full(170, n - 2), np.full(161, 300)]
    base = dags.random_dag(rng, n, 32, 8, bf, window=12)
    busy = dict(base, edge_src=np.concatenate([base["edge_src"]] + src).astype(np.int32),
                edge_dst=np.concatenate([base["edge_dst"]] + dst).astype(np.int32))
    graphs = [busy, dags.random_dag(rng, 90, 32, 8, bf), busy]
    b = dags.flatten(graphs, [0, 3], 2)
    b["model"] = dict(configs.MODEL[1], H=H, K=K, dtype=dtype, L=2, Hm=48, A_max=2)
    blob, _ = configs.make_weights(b["model"], 5, readout_scale=1.0 / 500.0)
    got = gpu_util.run_gpu(b, blob)
    want = xo.forward(b["model"], blob, b)
    assert got["status"] == 0
    gpu_util.assert_close(got["emb"], want["emb"], dtype, "graph_emb")
    gpu_util.assert_close(got["probs"], want["probs"], dtype, "probs")
    gpu_util.assert_close(got["value"], want["value"], dtype, "value")


def test_mask_beyond_candidates_raises_device_status():
    batch = configs.make_batch(1, candidates=5)
    blob, _ = gpu_util.default_weights(batch, 2)
    batch["mask"][0, 6] = 1
    got = gpu_util.run_gpu(batch, blob)
    assert got["status"] == 1
    assert got["probs"][0, 6] == 0.0


def test_results_are_bitwise_reproducible():
    batch = configs.make_batch(3, candidates=15)
    blob, _ = gpu_util.default_weights(batch, 4)
    a = gpu_util.run_gpu(batch, blob, sample=True, seed=3, step=9)
    b = gpu_util.run_gpu(batch, blob, sample=True, seed=3, step=9, where="device")
    for k in ("emb", "probs", "value", "action"):
        assert np.array_equal(a[k], b[k]), k


def test_bf16_model_takes_shape_features_off_the_bf16_grid(xo):
    """Section 3.3.2: shape features are arbitrary reals.  A bf16 model gets float32 features that are not
    bf16 values, graph by graph through xrl_pack; both sides round them to the storage type on their own."""
    import torch
    batch = configs.make_batch(3, candidates=7)
    m = batch["model"]
    rng = np.random.default_rng(12)
    batch["shape"] = (batch["shape"] + rng.uniform(1e-4, 3e-3, size=batch["shape"].shape)).astype(np.float32)
    assert not np.array_equal(batch["shape"], dags.round_to_bf16_grid(batch["shape"]))
    blob, _ = gpu_util.default_weights(batch, 1003)
    want = xo.forward(m, blob, batch)
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        ag.pack_graphs(dags.split(batch), batch["env_off"])
        o = ag.forward(torch.from_numpy(batch["mask"]).cuda())
        torch.cuda.synchronize()
        assert ag.device_status() == 0
        for k in ("emb", "probs", "value"):
            gpu_util.assert_close(o[k].cpu().numpy(), want[k], "bf16", k)
    finally:
        ag.close()

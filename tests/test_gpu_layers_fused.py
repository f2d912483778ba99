"""All attention layers of a small step in one cooperative launch (bf16, hidden 256, batches of at most
65,536 nodes) against the one-launch-per-layer path and against the oracle.  The two paths run the same
arithmetic in the same order, so their outputs must be equal bit for bit: node features after every
number of layers, graph embeddings, probabilities, values.  XRL_NO_FUSED_LAYERS=1 (read when a context
is created) selects the layer-by-layer path."""
import os

import numpy as np
import pytest

from workloads import configs
import gpu_util

pytestmark = pytest.mark.gpu


def _agent(batch, fused):
    old = os.environ.pop("XRL_NO_FUSED_LAYERS", None)
    if not fused:
        os.environ["XRL_NO_FUSED_LAYERS"] = "1"
    try:
        return gpu_util.make_agent(batch)
    finally:
        os.environ.pop("XRL_NO_FUSED_LAYERS", None)
        if old is not None:
            os.environ["XRL_NO_FUSED_LAYERS"] = old


def _both(batch, blob, layers_to_check=()):
    """Runs the batch on a fused and on a layer-by-layer context; returns (fused, plain) results, each with the
    step's outputs, the node features after the listed numbers of layers, and the encoder's launch count."""
    import torch
    import paper_2304_14698_b200 as xrl
    out = []
    for fused in (True, False):
        ag = _agent(batch, fused)
        try:
            res = gpu_util.run_gpu(batch, blob, where="device", agent=ag)
            assert res["status"] == 0
            res["launches"] = xrl.xrl_launch_counts(ag.ctx)["encode"]
            for nl in layers_to_check:
                res[("h", nl)] = xrl.xrl_debug_node_features(ag.ctx, ag.batch, nl, batch["model"]["H"])
            torch.cuda.synchronize()
            assert ag.device_status() == 0
            out.append(res)
        finally:
            ag.close()
    return out


def _check_equal(a, b, keys):
    for k in keys:
        assert np.array_equal(np.asarray(a[k]), np.asarray(b[k])), k


def test_paper_sized_step_equals_the_layer_by_layer_path_and_the_oracle(xo):
    batch = configs.make_batch(6)                       # 27 graphs, 15 k nodes, 5 layers: one tile per CTA
    L = batch["model"]["L"]
    blob, _ = gpu_util.default_weights(batch, 77)
    fused, plain = _both(batch, blob, layers_to_check=range(0, L + 1))
    _check_equal(fused, plain, ["emb", "probs", "value"] + [("h", nl) for nl in range(0, L + 1)])
    # pack + Eq. 6 + one launch for all layers + Eq. 8, against 2 L launches for the layers alone
    assert fused["launches"] <= 4 and plain["launches"] >= 2 * L + 2
    want = xo.forward(batch["model"], blob, batch)
    gpu_util.assert_close(fused["emb"], want["emb"], "bf16", "graph_emb")
    gpu_util.assert_close(fused["probs"], want["probs"], "bf16", "probs")
    gpu_util.assert_close(fused["value"], want["value"], "bf16", "value")
    nodes = xo.encode(batch["model"], blob, batch, want["packed"], dump_layer=L, want_nodes=True)["nodes"]
    gpu_util.assert_close(fused[("h", L)], nodes, "bf16", "node features after the last layer")


@pytest.mark.parametrize("candidates,nodes_scale", [(0, 0.05), (3, 0.01), (11, 1.0), (14, 1.0)])
def test_several_tiles_per_cta_ragged_last_tile_and_tiny_batches(xo, candidates, nodes_scale):
    # the power-law workload's model (hidden 256, 8 heads, 4 layers): from one graph of a few hundred nodes (a single
    # partly filled tile) to about 48 k / 60 k nodes (3 to 4 tiles per CTA, 16-row blocks in the attention phase)
    batch = configs.make_batch(4, candidates=candidates, nodes_scale=nodes_scale)
    N = int(batch["n_nodes"].sum())
    assert 0 < N <= 65536
    L = batch["model"]["L"]
    blob, _ = gpu_util.default_weights(batch, 5 + candidates)
    fused, plain = _both(batch, blob, layers_to_check=(1, L))
    _check_equal(fused, plain, ["emb", "probs", "value", ("h", 1), ("h", L)])
    assert fused["launches"] < plain["launches"]
    want = xo.forward(batch["model"], blob, batch)
    gpu_util.assert_close(fused["emb"], want["emb"], "bf16", "graph_emb")
    gpu_util.assert_close(fused["probs"], want["probs"], "bf16", "probs")


@pytest.mark.parametrize("K,L", [(4, 1), (8, 8), (8, 9), (4, 3)])
def test_other_head_counts_and_depths(xo, K, L):
    # 9 layers are more than the one-launch kernel takes: that context runs layer by layer (and still agrees)
    batch = configs.make_batch(6, candidates=5)
    m = dict(batch["model"], K=K, L=L)
    batch = dict(batch, model=m)
    blob, _ = configs.make_weights(m, 300 + L, readout_scale=1.0 / float(batch["n_nodes"].mean()))
    fused, plain = _both(batch, blob, layers_to_check=(L,))
    _check_equal(fused, plain, ["emb", "probs", "value", ("h", L)])
    if L <= 8:
        assert fused["launches"] < plain["launches"]
    else:
        assert fused["launches"] == plain["launches"]
    want = xo.forward(m, blob, batch)
    gpu_util.assert_close(fused["emb"], want["emb"], "bf16", "graph_emb")


def test_batches_above_the_size_limit_run_layer_by_layer():
    import paper_2304_14698_b200 as xrl
    batch = configs.make_batch(4, candidates=19)        # about 80 k nodes
    assert int(batch["n_nodes"].sum()) > 65536
    blob, _ = gpu_util.default_weights(batch, 9)
    ag = _agent(batch, True)
    try:
        res = gpu_util.run_gpu(batch, blob, where="device", agent=ag)
        assert res["status"] == 0
        assert xrl.xrl_launch_counts(ag.ctx)["encode"] >= 2 * batch["model"]["L"] + 2
    finally:
        ag.close()

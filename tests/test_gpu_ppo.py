"""GPU parity of the training step's gradient (Section 3.3.4, Eq. 3-5): the loss terms, the log-probabilities
and the gradient with respect to every weight tensor against the oracle's reverse pass."""
import numpy as np
import pytest

from workloads import configs, dags
import gpu_util
from test_gpu_fuzz import _random_case

pytestmark = pytest.mark.gpu

# Per weight tensor: |g - r| <= a max|r| + b |r| for every entry, and ||g - r||_2 <= c ||r||_2 + d ||r_all||_2.
# "fp32" is the check of the reverse pass itself, against the definition.
# "bf16": a bf16 model keeps Z and every layer's output in bf16 while the definition keeps them exact, so each
# term of a gradient sum is off by a fraction of a percent per layer it passed.  The pass criterion is still the
# definition.  Entry by entry: the encoder's matrices and biases (W0, b0, W_l, b_l) within 12 % and the value
# head within 5 % of the tensor's largest entry (largest observed over the cases below: 10 % and 3 %).  By norms
# only (15 % of the tensor's own norm plus 1 % of the whole gradient's): Eq. 8 (W_g, b_g) and the policy head,
# where one hidden unit of one graph whose pre-activation sits within rounding of zero lands on the other side
# of its ReLU and moves that unit's whole column (batches here have 10-30 graphs), and the attention vectors
# a_src / a_dst, whose gradients are sums of cancelling terms of size 1e-4 that show the rounding of Z as a
# large part of their own, small, norm.
# "bf16 mirrored" (a debugging aid, not the criterion): against the oracle run at the rounded activations, with
# the half-scores taken where the transform kernel of that shape takes them, what remains are values that fall on
# the other side of a rounding boundary or of a ReLU's zero.
GRAD_TOL = {"fp32": (1e-3, 1e-3, 1e-3, 0.0), "bf16 mirrored": (3e-2, 2e-2, 3e-2, 0.0),
            "bf16": (None, 0.0, 0.15, 0.01)}
# entry-by-entry bounds of a bf16 model against the definition, by tensor-name prefix (fraction of the largest entry)
BF16_ENTRYWISE = {"W0": 0.12, "b0": 0.12, "W1": 0.12, "W2": 0.12, "W3": 0.12, "W4": 0.12, "W5": 0.12,
                  "b1": 0.12, "b2": 0.12, "b3": 0.12, "b4": 0.12, "b5": 0.12,
                  "vW1": 0.05, "vb1": 0.05, "vWh": 0.05, "vbh": 0.05, "vw2": 0.05}


def _check_grad(m, got, want, tol, what, entrywise=None):
    off = 0
    nall = float(np.linalg.norm(want))
    for name, shape in configs.weight_layout(m):
        n = int(np.prod(shape))
        off += n
        if n == 0:
            continue
        g, r = got[off - n:off], want[off - n:off]
        # pb2's gradient is exactly 0 (the softmax ignores a shift of all logits): the GPU's is a sum of fp32 roundings
        floor = 1e-5 if np.abs(r).max() < 1e-12 else 1e-6
        frac = tol[0] if entrywise is None else entrywise.get(name)
        if frac is not None:
            bound = frac * np.abs(r).max() + tol[1] * np.abs(r) + floor
            err = np.abs(g - r)
            if (err > bound).any():
                i = int(np.argmax(err - bound))
                raise AssertionError(f"{what} {name}: {(err > bound).sum()} of {n} outside tolerance; worst at {i}: "
                                     f"got {g[i]!r} want {r[i]!r} (max |want| {np.abs(r).max():.3e})")
        nerr, nref = float(np.linalg.norm(g - r)), float(np.linalg.norm(r))
        assert nerr <= tol[2] * nref + tol[3] * nall + floor, \
            f"{what} {name}: ||g - r|| = {nerr:.3e}, ||r|| = {nref:.3e}, ||r_all|| = {nall:.3e}"
    if tol[3] > 0:
        assert np.linalg.norm(got - want) <= 0.15 * nall, (what, float(np.linalg.norm(got - want)), nall)

def _transitions(xo, m, blob, batch, packed, seed, g0=None):
    """Actions, old log-probabilities, advantages and value targets for every environment of the batch."""
    rng = np.random.default_rng(seed)
    enc = xo.encode(m, blob, batch, packed, g0=g0)
    st, _, probs, _ = xo.policy_value(m, blob, batch, enc["emb"])
    assert st == 0
    ne = probs.shape[0]
    action = np.array([rng.choice(np.flatnonzero(probs[e] > 0)) for e in range(ne)], np.int32)
    logp_now = np.log(probs[np.arange(ne), action])
    # ratios on both sides of the clipping range and inside it
    logp_old = logp_now + rng.choice([-0.5, -0.05, 0.03, 0.4], size=ne)
    adv = rng.normal(size=ne)
    ret = rng.normal(size=ne)
    return action, logp_old, adv, ret


def _compare(xo, batch, m, blob, g0=None, seed=0, eps=0.2, c1=0.5, c2=0.01, mirrored=True):
    import torch
    import paper_2304_14698_b200 as xrl
    st, packed = xo.pack(batch)
    assert st == 0
    action, logp_old, adv, ret = _transitions(xo, m, blob, batch, packed, seed, g0)
    want = xo.ppo_grad(m, blob, batch, packed, action, logp_old, adv, ret, eps, c1, c2, g0=g0)
    ag = gpu_util.make_agent(batch, slack=2)
    try:
        ag.set_weights(blob)
        ag.pack(batch)
        f32 = lambda a: torch.from_numpy(np.asarray(a, np.float32)).cuda()
        loss = torch.full((4,), 7.0, device="cuda")
        grad = torch.full((len(blob),), 7.0, device="cuda")
        logp = torch.empty(len(action), device="cuda")
        g0d = None if g0 is None else f32(g0)
        for _ in range(2):                 # the second call reuses the workspace and must overwrite, not add
            xrl.xrl_ppo_grad(ag.ctx, ag.batch, torch.from_numpy(batch["mask"]).cuda(),
                             torch.from_numpy(action).cuda(), f32(logp_old), f32(adv), f32(ret), loss, grad,
                             eps=eps, c1=c1, c2=c2, g0=g0d, logp_out=logp)
        torch.cuda.synchronize()
        assert ag.device_status() == 0
        dt = m["dtype"]
        gpu_util.assert_close(loss.cpu().numpy(), want["loss"], dt, "loss")
        gpu_util.assert_close(logp.cpu().numpy(), want["logp"], dt, "logp")
        got = grad.cpu().numpy().astype(np.float64)
        _check_grad(m, got, want["grad"], GRAD_TOL[dt], "definition",
                    entrywise=BF16_ENTRYWISE if dt == "bf16" else None)
        if dt == "bf16" and mirrored:
            mir = xo.ppo_grad(m, blob, batch, packed, action, logp_old, adv, ret, eps, c1, c2, g0=g0,
                              mirrored=1 if m["H"] in (128, 256) else 2)
            _check_grad(m, got, mir["grad"], GRAD_TOL["bf16 mirrored"], "mirrored")
            np.testing.assert_allclose(loss.cpu().numpy(), mir["loss"], rtol=2e-3, atol=1e-4)
        # the forward pass of the same context still works afterwards and agrees with the oracle
        o = ag.forward(torch.from_numpy(batch["mask"]).cuda(), g0=g0d)
        torch.cuda.synchronize()
        enc = xo.encode(m, blob, batch, packed, g0=g0)
        gpu_util.assert_close(o["emb"].cpu().numpy(), enc["emb"], dt, "emb after the gradient")
    finally:
        ag.close()


def _small_batch(m, seed, envs=(3, 0, 5), nodes=(3, 40), edge_attr=False):
    rng = dags.make_rng(seed)
    graphs, env_off = [], [0]
    for c in envs:
        for _ in range(c + 1):
            graphs.append(dags.random_dag(rng, int(rng.integers(*nodes)), m["T"], 8, m["dtype"] == "bf16", window=6))
        env_off.append(len(graphs))
    b = dags.flatten(graphs, env_off, m["A_max"])
    b["mask"][0, 1] = 0
    if edge_attr:
        b["edge_attr"] = dags.tensor_shape_attributes(rng, int(b["n_edges"].sum()), 8, m["dtype"] == "bf16")
    b["model"] = m
    return b


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("variant", ["plain", "two hidden layers", "edge attributes", "both ways", "no layers",
                                     "three heads", "hidden 256"])
def test_gradient_matches_the_oracle(xo, dtype, variant):
    m = dict(T=12, S=8, H=64, K=4, L=2, Hm=24, Dg=2, dtype=dtype, A_max=6)
    if variant == "two hidden layers":
        m["Hm2"] = 9
    if variant == "edge attributes":
        m["edge_attr"] = True
    if variant == "both ways":
        m["both_ways"] = True
    if variant == "no layers":
        m["L"] = 0
    if variant == "three heads":
        m.update(H=96, K=3, L=1)
    if variant == "hidden 256":                      # the tensor-core transform and merged Z rows (bf16)
        m.update(H=256, K=8, L=3, Hm=64, Hm2=16, T=40)
    b = _small_batch(m, 11, edge_attr=(variant == "edge attributes"))
    blob, _ = gpu_util.default_weights(b, 5)
    rng = np.random.default_rng(2)
    g0 = rng.normal(size=(b["num_graphs"], m["Dg"]))
    _compare(xo, b, m, blob, g0=g0, seed=3)


@pytest.mark.parametrize("seed", range(16))
def test_gradient_on_random_batches(xo, seed):
    batch, m, blob, _hint, g0 = _random_case(seed)
    _compare(xo, batch, m, blob, g0=g0, seed=seed)


def test_gradient_on_a_step_of_the_papers_size(xo):
    b = configs.make_batch(6, candidates=5)
    blob, _ = gpu_util.default_weights(b, 1)
    _compare(xo, b, b["model"], blob, seed=4)


def test_gradient_on_many_rows_of_the_large_step(xo):
    """128 k rows of the power-law workload at hidden 256 in bf16: the tensor-core products of the reverse pass
    run many tiles per CTA and the reverse attention kernel sees the workload's fan-out."""
    b = configs.make_batch(4, candidates=31)
    assert int(b["n_nodes"].sum()) > 100_000
    blob, _ = gpu_util.default_weights(b, 2)
    _compare(xo, b, b["model"], blob, seed=6, mirrored=False)     # (one run of the oracle's reverse pass: ~2 min)


def test_gradient_exchange_weights_on_the_device():
    """xrl_grad_weigh / xrl_grad_unweigh on device buffers: buf = [grad n | loss n | n], then grad, loss = buf /
    buf[-1] (here after adding a second rank's buffer by hand)."""
    import torch
    import paper_2304_14698_b200 as xrl
    rng = np.random.default_rng(3)
    for dtype in (torch.float32, torch.float64):
        g1, g2 = rng.normal(size=1000), rng.normal(size=1000)
        l1, l2 = rng.normal(size=4), rng.normal(size=4)
        bufs = []
        for g, l, n in ((g1, l1, 3), (g2, l2, 5)):
            gd, ld = torch.tensor(g, dtype=dtype, device="cuda"), torch.tensor(l, dtype=dtype, device="cuda")
            buf = torch.empty(1005, dtype=dtype, device="cuda")
            xrl.xrl_grad_weigh(gd, ld, n, buf)
            bufs.append(buf)
        total_buf = bufs[0] + bufs[1]                       # what a sum all-reduce leaves on every rank
        gd, ld = torch.empty(1000, dtype=dtype, device="cuda"), torch.empty(4, dtype=dtype, device="cuda")
        assert xrl.xrl_grad_unweigh(total_buf, gd, ld) == 8
        tol = 1e-6 if dtype == torch.float32 else 1e-14
        np.testing.assert_allclose(gd.cpu().numpy(), (3 * g1 + 5 * g2) / 8, rtol=tol, atol=tol)
        np.testing.assert_allclose(ld.cpu().numpy(), (3 * l1 + 5 * l2) / 8, rtol=tol, atol=tol)


def test_an_action_the_mask_excludes_is_reported(xo):
    import torch
    import paper_2304_14698_b200 as xrl
    m = dict(T=12, S=8, H=64, K=4, L=1, Hm=24, Dg=0, dtype="fp32", A_max=6)
    b = _small_batch(m, 1)
    blob, _ = gpu_util.default_weights(b, 5)
    ag = gpu_util.make_agent(b)
    try:
        ag.set_weights(blob)
        ag.pack(b)
        ne = len(b["env_off"]) - 1
        z = torch.zeros(ne, device="cuda")
        action = torch.full((ne,), m["A_max"], dtype=torch.int32, device="cuda")
        action[0] = 1                                   # masked out in _small_batch
        loss = torch.empty(4, device="cuda"); grad = torch.empty(len(blob), device="cuda")
        xrl.xrl_ppo_grad(ag.ctx, ag.batch, torch.from_numpy(b["mask"]).cuda(), action, z, z, z, loss, grad)
        assert ag.device_status() == 1
        with pytest.raises(xrl.XrlError) as e:
            xrl.xrl_ppo_grad(ag.ctx, ag.batch, torch.from_numpy(b["mask"]).cuda(), action, z, z, z, None, grad)
        assert e.value.status == 1
        # not recordable: inside a recording bracket the call is refused and nothing is enqueued
        mask_d = torch.from_numpy(b["mask"]).cuda()     # (copies are not allowed inside the bracket)
        torch.cuda.synchronize()
        xrl.xrl_graph_begin(ag.ctx)
        with pytest.raises(xrl.XrlError) as e:
            xrl.xrl_ppo_grad(ag.ctx, ag.batch, mask_d, action, z, z, z, loss, grad)
        assert xrl.STATUS_NAMES[e.value.status] == "XRL_ERR_STATE"
        try:
            xrl.xrl_graph_launch(ag.ctx)            # ends the (empty) recording
        except xrl.XrlError:
            pass
    finally:
        ag.close()


def test_advantage_estimates_match_the_oracle(xo):
    import torch
    import paper_2304_14698_b200 as xrl
    rng = np.random.default_rng(9)
    T, M = 37, 203
    reward = rng.normal(size=(T, M)); values = rng.normal(size=(T + 1, M))
    done = (rng.random((T, M)) < 0.1).astype(np.uint8)
    done[:, 0] = 0; done[:, 1] = 1                      # a trajectory that never ends, one that ends every step
    f32 = lambda a: torch.from_numpy(np.asarray(a, np.float32)).cuda()
    for gamma, lam in ((0.99, 0.95), (1.0, 1.0), (0.9, 0.0)):
        adv, ret = xrl.xrl_gae(f32(reward), f32(values), torch.from_numpy(done).cuda(), gamma, lam)
        torch.cuda.synchronize()
        for j in (0, 1, 2, 57, M - 1):
            a, r = xo.gae(reward[:, j].astype(np.float32), values[:, j].astype(np.float32), done[:, j], gamma, lam)
            gpu_util.assert_close(adv[:, j].cpu().numpy(), a, "fp32", f"adv {j}")
            gpu_util.assert_close(ret[:, j].cpu().numpy(), r, "fp32", f"ret {j}")
    a0, r0 = xrl.xrl_gae(torch.empty((0, 5), device="cuda"), torch.empty((1, 5), device="cuda"),
                         torch.empty((0, 5), dtype=torch.uint8, device="cuda"), 0.9, 0.9)
    assert a0.shape == (0, 5)


def test_gradient_of_a_batch_packed_range_by_range(xo, monkeypatch):
    """The gradient call joins the ranges of a batch that was copied and packed range by range."""
    import torch
    import paper_2304_14698_b200 as xrl
    from test_gpu_pipeline import _pinned, _pack_pinned
    monkeypatch.setenv("XRL_PIPELINE_MIN_NODES", "2000")
    batch = configs.make_batch(3, candidates=15)
    m = batch["model"]
    blob, _ = gpu_util.default_weights(batch, 8)
    st, packed = xo.pack(batch)
    assert st == 0
    action, logp_old, adv, ret = _transitions(xo, m, blob, batch, packed, 1)
    mir = xo.ppo_grad(m, blob, batch, packed, action, logp_old, adv, ret, mirrored=1)
    ag = gpu_util.make_agent(batch)
    try:
        ag.set_weights(blob)
        keep = _pinned(ag, batch)
        _pack_pinned(xrl, ag, batch, keep)
        f32 = lambda a: torch.from_numpy(np.asarray(a, np.float32)).cuda()
        loss = torch.empty(4, device="cuda"); grad = torch.empty(len(blob), device="cuda")
        xrl.xrl_ppo_grad(ag.ctx, ag.batch, torch.from_numpy(batch["mask"]).cuda(), torch.from_numpy(action).cuda(),
                         f32(logp_old), f32(adv), f32(ret), loss, grad)
        torch.cuda.synchronize()
        assert ag.device_status() == 0
        _check_grad(m, grad.cpu().numpy().astype(np.float64), mir["grad"], GRAD_TOL["bf16 mirrored"], "mirrored")
    finally:
        ag.close()

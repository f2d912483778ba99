"""Helpers shared by the GPU parity tests: run a workload through the C-ABI library."""
import numpy as np

from workloads import configs

TOL = {"fp32": (1e-4, 1e-3), "bf16": (2e-2, 2e-2)}      # (atol, rtol): |x - r| <= atol + rtol |r|


def assert_close(got, want, dtype, what=""):
    atol, rtol = TOL[dtype]
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    err = np.abs(got - want)
    bound = atol + rtol * np.abs(want)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: "
                             f"got {got[i]!r} want {want[i]!r} (|err| {err[i]:.3e}, bound {bound[i]:.3e})")


def make_agent(batch, m=None, slack=0):
    import paper_2304_14698_b200 as xrl
    m = dict(batch["model"] if m is None else m)
    N = int(batch["n_nodes"].sum()); E = int(batch["n_edges"].sum())
    return xrl.Agent(m, batch["num_graphs"] + slack, len(batch["env_off"]) - 1 + slack,
                     max(1, N + slack), max(1, E + slack))


def default_weights(batch, seed, **kw):
    m = batch["model"]
    scale = 1.0 / max(1.0, float(batch["n_nodes"].mean()))
    return configs.make_weights(m, seed, readout_scale=kw.pop("readout_scale", scale), **kw)


def run_gpu(batch, blob, sample=False, seed=0, step=0, where="host", agent=None):
    import torch
    own = agent is None
    ag = make_agent(batch) if own else agent
    try:
        ag.set_weights(blob)
        if where == "host":
            ag.pack(batch)
        else:
            dev = {k: batch[k] for k in ("n_nodes", "n_edges", "env_off")}
            dev["op"] = torch.from_numpy(batch["op"]).cuda()
            shp = torch.from_numpy(batch["shape"]).cuda()
            dev["shape"] = shp.to(torch.bfloat16) if batch["model"]["dtype"] == "bf16" else shp
            dev["edge_src"] = torch.from_numpy(batch["edge_src"]).cuda()
            dev["edge_dst"] = torch.from_numpy(batch["edge_dst"]).cuda()
            ag.pack(dev)
        mask = torch.from_numpy(batch["mask"]).cuda()
        o = ag.forward(mask, sample=sample, seed=seed, step=step)
        torch.cuda.synchronize()
        res = {k: v.cpu().numpy() for k, v in o.items()}
        res["status"] = ag.device_status()
        return res
    finally:
        if own:
            ag.close()

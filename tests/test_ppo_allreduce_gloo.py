"""The data-parallel training step's exchange on CPU: two gloo ranks each hold the gradient of the PPO
objective over their own environments (here from the oracle, in float64); after the weighted all-reduce both
hold the gradient over all environments, equal to the oracle's on the whole batch."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    sys.path.insert(0, os.path.join(%r, "tests"))
    import numpy as np, torch, torch.distributed as dist
    from workloads import configs, dags
    from oracle import xrl_oracle as xo
    import paper_2304_14698_b200 as xrl
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    m = dict(T=6, S=8, H=16, K=2, L=2, Hm=8, Dg=0, dtype="fp32", A_max=4)
    rng = dags.make_rng(7)
    envs = [3, 1, 4]                         # candidates per environment; rank 0 takes the first, rank 1 the rest
    graphs = [[dags.random_dag(rng, int(rng.integers(3, 12)), m["T"], 8, False, window=4) for _ in range(c + 1)]
              for c in envs]
    def batch_of(ids):
        gs, off = [], [0]
        for e in ids:
            gs += graphs[e]; off.append(len(gs))
        b = dags.flatten(gs, off, m["A_max"]); b["model"] = m
        return b
    blob, _ = configs.make_weights(m, 3, readout_scale=0.3)
    blob = blob.astype(np.float32)
    action = np.array([1, 4, 0], np.int32); logp_old = np.array([-1.2, -0.4, -1.9])
    adv = np.array([0.5, -1.0, 2.0]); ret = np.array([0.1, 0.2, -0.3])
    def grad_of(ids):
        b = batch_of(ids)
        st, packed = xo.pack(b); assert st == 0
        ids = np.asarray(ids)
        return xo.ppo_grad(m, blob, b, packed, action[ids], logp_old[ids], adv[ids], ret[ids])
    mine = [0] if rank == 0 else [1, 2]
    g = grad_of(mine)
    grad = torch.from_numpy(g["grad"].copy()); loss = torch.from_numpy(g["loss"].copy())
    total = xrl.allreduce_ppo_grad(loss, grad, len(mine))
    whole = grad_of([0, 1, 2])
    ok = (total == 3 and np.allclose(grad.numpy(), whole["grad"], rtol=1e-12, atol=1e-14)
          and np.allclose(loss.numpy(), whole["loss"], rtol=1e-12, atol=1e-14)
          and not np.allclose(g["grad"], whole["grad"], rtol=1e-3))
    flags = [None, None]
    dist.all_gather_object(flags, bool(ok))
    if rank == 0:
        print(json.dumps({"ok": flags}))
    dist.destroy_process_group()
""") % (ROOT, ROOT)


def test_weighted_gradient_allreduce_equals_the_whole_batch(tmp_path, xo):
    script = tmp_path / "ranks.py"
    script.write_text(SCRIPT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29613", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600,
                       env=dict(os.environ, CUDA_VISIBLE_DEVICES=""))
    assert r.returncode == 0, r.stderr[-3000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    assert json.loads(line)["ok"] == [True, True]

"""The five benchmark workloads (and reduced variants of them) as seeded synthetic batches,
plus seeded weight blobs.  No arithmetic of the encoded method lives here.

model config keys: T (operator types), S (shape features), H (hidden), K (heads),
L (graph-attention layers), Hm (MLP hidden), Dg (global attribute width),
dtype ("fp32" | "bf16"), A_max (padded candidate slots); optional Hm2 (second MLP hidden width).

Workload 6 is not one of the benchmark's five: it carries the values of the paper's hyper-parameter
table (5 attention layers, MLP heads with hidden sizes [256, 64], about 40 operator types) on a step
of the size its workload table reports for BERT (26 candidates of a transformer-shaped graph).
"""
from __future__ import annotations

import numpy as np

from . import dags

MODEL = {
    1: dict(T=32, S=8, H=64, K=1, L=2, Hm=64, Dg=1, dtype="fp32", A_max=8),
    2: dict(T=32, S=8, H=128, K=4, L=3, Hm=128, Dg=1, dtype="fp32", A_max=64),
    3: dict(T=32, S=8, H=128, K=4, L=3, Hm=128, Dg=1, dtype="bf16", A_max=256),
    4: dict(T=64, S=8, H=256, K=8, L=4, Hm=256, Dg=1, dtype="bf16", A_max=1024),
    5: dict(T=64, S=8, H=256, K=8, L=4, Hm=256, Dg=1, dtype="bf16", A_max=128),
    6: dict(T=40, S=8, H=256, K=8, L=5, Hm=256, Hm2=64, Dg=1, dtype="bf16", A_max=32),
}
# candidates per environment and number of environments at full size
FULL = {1: (7, 1), 2: (63, 1), 3: (255, 1), 4: (1023, 1), 5: (127, 64), 6: (26, 1)}
NAME = {1: "tiny_step", 2: "transformer_step", 3: "cnn_step", 4: "large_step", 5: "rollout_batch",
        6: "paper_step"}


def _base_graph(cfg_id, rng, env, m, nodes_scale=1.0):
    bf16 = m["dtype"] == "bf16"
    if cfg_id == 1:
        return dags.random_dag(rng, 64, m["T"], m["S"], bf16)
    if cfg_id in (2, 6):
        return dags.transformer_dag(rng, 12, 3, m["T"], m["S"], bf16)
    if cfg_id == 3:
        return dags.cnn_dag(rng, int(1200 * nodes_scale), m["T"], m["S"], bf16)
    if cfg_id == 4:
        return dags.powerlaw_dag(rng, int(4000 * nodes_scale), m["T"], m["S"], bf16)
    if env % 2 == 0:      # rollout batch: transformer-like and CNN-like environments alternate
        return dags.transformer_dag(rng, 12, 6, m["T"], m["S"], bf16)
    return dags.cnn_dag(rng, 1000, m["T"], m["S"], bf16)


def make_batch(cfg_id, candidates=None, envs=None, seed=None, mask_fraction=None,
               nodes_scale=1.0):
    """Build workload `cfg_id`.  `candidates` / `envs` shrink it (graph sizes and model
    dimensions unchanged) so that a slow CPU implementation can check every output."""
    m = MODEL[cfg_id]
    c_full, e_full = FULL[cfg_id]
    C = c_full if candidates is None else int(candidates)
    Ne = e_full if envs is None else int(envs)
    rng = dags.make_rng(cfg_id if seed is None else seed)
    bf16 = m["dtype"] == "bf16"
    graphs, env_off = [], [0]
    for e in range(Ne):
        cur = _base_graph(cfg_id, rng, e, m, nodes_scale)
        graphs.append(cur)
        for _ in range(C):
            if cfg_id == 1:    # independent DAGs
                graphs.append(dags.random_dag(rng, 64, m["T"], m["S"], bf16))
            else:
                graphs.append(dags.local_rewrite(rng, cur, m["T"], bf16))
        env_off.append(len(graphs))
    A = m["A_max"]
    mask = np.zeros((Ne, A), dtype=np.uint8)
    frac = (0.01 if cfg_id == 4 else 0.0) if mask_fraction is None else mask_fraction
    for e in range(Ne):
        c = min(C, A)
        mask[e, :c] = 1
        if frac > 0 and c > 1:
            drop = rng.random(c) < frac
            mask[e, :c][drop] = 0
    batch = dags.flatten(graphs, env_off, A, mask)
    batch["model"] = dict(m)
    batch["name"] = NAME[cfg_id]
    return batch


# ----------------------------------------------------------------------------------------
# weights: one flat float32 blob, matrices row-major [in x out], in this order
#   W0 [(S+T+S) x H], b0 [H]
#   per layer: W [H x H], a_src [H], a_dst [H], b [H]
#   Wg [(H+Dg) x H], bg [H]
#   policy: W1 [H x Hm], b1 [Hm], (Wh [Hm x Hm2], bh [Hm2] if Hm2 > 0), w2 [last hidden], b2 [1]
#   value : W1 [2H x Hm], b1 [Hm], (Wh [Hm x Hm2], bh [Hm2] if Hm2 > 0), w2 [last hidden], b2 [1]
def weight_layout(m):
    S, T, H, K, L, Hm, Dg = m["S"], m["T"], m["H"], m["K"], m["L"], m["Hm"], m["Dg"]
    Hm2 = int(m.get("Hm2", 0))
    last = Hm2 if Hm2 > 0 else Hm
    second = lambda p: [(p + "Wh", (Hm, Hm2)), (p + "bh", (Hm2,))] if Hm2 > 0 else []
    items = [("W0", (2 * S + T, H)), ("b0", (H,))]
    for l in range(L):
        items += [(f"W{l + 1}", (H, H)), (f"a_src{l + 1}", (H,)), (f"a_dst{l + 1}", (H,)),
                  (f"b{l + 1}", (H,))]
    items += [("Wg", (H + Dg, H)), ("bg", (H,)),
              ("pW1", (H, Hm)), ("pb1", (Hm,))] + second("p") + [("pw2", (last,)), ("pb2", (1,)),
              ("vW1", (2 * H, Hm)), ("vb1", (Hm,))] + second("v") + [("vw2", (last,)), ("vb2", (1,))]
    return items


def weight_count(m):
    return int(sum(int(np.prod(s)) for _, s in weight_layout(m)))


def make_weights(m, seed, readout_scale=1.0, zero_attention=False):
    """Xavier-uniform matrices and attention vectors, biases U(-0.1, 0.1).
    `readout_scale` multiplies Wg's readout rows (a sum over thousands of nodes would
    otherwise saturate every later softmax)."""
    rng = dags.make_rng(seed)
    d = m["H"] // m["K"]
    parts = {}
    for name, shp in weight_layout(m):
        if len(shp) == 2:
            bound = np.sqrt(6.0 / (shp[0] + shp[1]))
            w = rng.uniform(-bound, bound, size=shp)
        elif name.startswith("a_"):
            bound = np.sqrt(6.0 / (d + 1))
            w = rng.uniform(-bound, bound, size=shp)
            if zero_attention:
                w[:] = 0.0
        elif name.endswith("w2"):
            bound = np.sqrt(6.0 / (shp[0] + 1))
            w = rng.uniform(-bound, bound, size=shp)
        else:
            w = rng.uniform(-0.1, 0.1, size=shp)
        if name == "Wg":
            w[: m["H"]] *= readout_scale
        parts[name] = w.astype(np.float32)
    blob = np.concatenate([parts[n].ravel() for n, _ in weight_layout(m)]).astype(np.float32)
    return blob, parts


def unpack_weights(m, blob):
    out, off = {}, 0
    for name, shp in weight_layout(m):
        cnt = int(np.prod(shp))
        out[name] = blob[off:off + cnt].reshape(shp)
        off += cnt
    assert off == len(blob)
    return out


def pack_weights(m, parts):
    return np.concatenate([np.asarray(parts[n], dtype=np.float32).ravel()
                           for n, _ in weight_layout(m)]).astype(np.float32)

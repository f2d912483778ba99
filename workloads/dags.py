"""Seeded synthetic computation DAGs shaped like the graphs the agent observes.

Holds no arithmetic of the encoded method: only graph structure, operator ids,
shape features, masks.  Both the CPU oracle's tests and the CUDA library's tests
draw their inputs from here, so that the two sides see identical bytes.

A graph is a dict of numpy arrays:
    op        int32  [n]      operator id in [0, T)
    shape     float32[n, S]   shape features in [0, 1]
    edge_src  int32  [m]      producer (local id)
    edge_dst  int32  [m]      consumer (local id)
Nodes are emitted in a topological order (every edge goes from a lower to a
higher id), which makes acyclicity hold by construction.

The structure follows the paper's description of its observations (Section 3.3.1
and 3.3.2: the current graph plus a list of candidates, each obtained by one
rewrite at one location) -- the real graphs come from a rewrite engine that is not
available, so local random rewrites stand in for them.
"""
from __future__ import annotations

import numpy as np

# A small operator table (the paper's table has about forty tensor operators, Section 3.3.2).
OP_INPUT, OP_WEIGHT, OP_MATMUL, OP_ADD, OP_SOFTMAX, OP_LAYERNORM, OP_TRANSPOSE, \
    OP_RESHAPE, OP_SCALE, OP_GELU, OP_CONV, OP_BATCHNORM, OP_RELU, OP_CONCAT, \
    OP_SPLIT, OP_POOL = range(16)


def make_rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed)))


def round_to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16-representable float32 (ties to even)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def shape_features(rng: np.random.Generator, n: int, S: int, bf16: bool) -> np.ndarray:
    """log2(dim)/12 with dim log-uniform in [1, 4096]: S numbers in [0, 1] per node."""
    dim = np.floor(np.exp2(12.0 * rng.random((n, S)))).clip(1, 4096)
    f = (np.log2(dim) / 12.0).astype(np.float32)
    return round_to_bf16_grid(f) if bf16 else f


def _finish(ops, src, dst, rng, S, bf16):
    n = len(ops)
    return {
        "op": np.asarray(ops, dtype=np.int32),
        "shape": shape_features(rng, n, S, bf16),
        "edge_src": np.asarray(src, dtype=np.int32),
        "edge_dst": np.asarray(dst, dtype=np.int32),
    }


def random_dag(rng, n=64, T=32, S=8, bf16=False, window=16):
    """Node i draws in-degree min(i, Binomial(4, 1/2)); predecessors without
    replacement from the previous `window` nodes."""
    src, dst = [], []
    for i in range(1, n):
        lo = max(0, i - window)
        k = min(i - lo, int(rng.binomial(4, 0.5)))
        if k:
            for p in rng.choice(np.arange(lo, i), size=k, replace=False):
                src.append(int(p)); dst.append(i)
    ops = rng.integers(0, T, size=n)
    return _finish(ops, src, dst, rng, S, bf16)


class _Builder:
    def __init__(self):
        self.ops, self.src, self.dst = [], [], []

    def node(self, op, *inputs):
        i = len(self.ops)
        self.ops.append(op)
        for p in inputs:
            self.src.append(p); self.dst.append(i)
        return i


def transformer_dag(rng, blocks=12, heads=3, T=32, S=8, bf16=False):
    """Encoder blocks written out as operator nodes, attention heads unrolled."""
    b = _Builder()
    x = b.node(OP_INPUT)
    pos = b.node(OP_WEIGHT)
    x = b.node(OP_ADD, x, pos)
    x = b.node(OP_LAYERNORM, x)
    for _ in range(blocks):
        xin = b.node(OP_RESHAPE, x)
        ctx = []
        for _h in range(heads):
            q = b.node(OP_MATMUL, xin, b.node(OP_WEIGHT))
            k = b.node(OP_MATMUL, xin, b.node(OP_WEIGHT))
            v = b.node(OP_MATMUL, xin, b.node(OP_WEIGHT))
            kt = b.node(OP_TRANSPOSE, k)
            s = b.node(OP_MATMUL, q, kt)
            s = b.node(OP_SCALE, s)
            p = b.node(OP_SOFTMAX, s)
            ctx.append(b.node(OP_MATMUL, p, v))
        c = b.node(OP_CONCAT, *ctx)
        c = b.node(OP_RESHAPE, c)
        o = b.node(OP_MATMUL, c, b.node(OP_WEIGHT))
        x = b.node(OP_LAYERNORM, b.node(OP_ADD, x, o))
        f = b.node(OP_MATMUL, x, b.node(OP_WEIGHT))
        f = b.node(OP_GELU, f)
        f = b.node(OP_MATMUL, f, b.node(OP_WEIGHT))
        x = b.node(OP_LAYERNORM, b.node(OP_ADD, x, f))
    b.node(OP_MATMUL, x, b.node(OP_WEIGHT))
    return _finish(b.ops, b.src, b.dst, rng, S, bf16)


def cnn_dag(rng, target_nodes=1200, T=32, S=8, bf16=False):
    """Residual convolution blocks with 1..4 parallel branches joined by a concat."""
    b = _Builder()
    x = b.node(OP_INPUT)
    x = b.node(OP_RELU, b.node(OP_BATCHNORM, b.node(OP_CONV, x, b.node(OP_WEIGHT))))
    x = b.node(OP_POOL, x)
    while len(b.ops) < target_nodes - 40:
        nb = int(rng.integers(1, 5))
        depth = int(rng.integers(1, 4))
        outs = []
        for _ in range(nb):
            y = x
            for _d in range(depth):
                y = b.node(OP_CONV, y, b.node(OP_WEIGHT))
                y = b.node(OP_BATCHNORM, y)
                y = b.node(OP_RELU, y)
            outs.append(y)
        y = b.node(OP_CONCAT, *outs) if nb > 1 else outs[0]
        y = b.node(OP_BATCHNORM, b.node(OP_CONV, y, b.node(OP_WEIGHT)))
        x = b.node(OP_RELU, b.node(OP_ADD, x, y))
        if rng.random() < 0.15:
            x = b.node(OP_POOL, x)
    x = b.node(OP_POOL, x)
    b.node(OP_MATMUL, x, b.node(OP_WEIGHT))
    return _finish(b.ops, b.src, b.dst, rng, S, bf16)


def powerlaw_dag(rng, n=4000, T=64, S=8, bf16=False, alpha=2.2, kmax=64, window=256):
    """Out-degree k with P(k) ~ k^-alpha on 1..kmax, consumers among the next `window` ids."""
    ks = np.arange(1, kmax + 1, dtype=np.float64)
    pk = ks ** (-alpha)
    pk /= pk.sum()
    deg = rng.choice(np.arange(1, kmax + 1), size=n, p=pk)
    src, dst = [], []
    for i in range(n - 1):
        hi = min(n - 1, i + window)
        k = min(int(deg[i]), hi - i)
        t = rng.choice(np.arange(i + 1, hi + 1), size=k, replace=False)
        src.extend([i] * k); dst.extend(int(v) for v in t)
    ops = rng.integers(0, T, size=n)
    return _finish(ops, src, dst, rng, S, bf16)


def local_rewrite(rng, g, T, bf16=False, max_region=6, max_new=6):
    """One candidate: replace a run of 2..max_region consecutive (hence convex) nodes by
    1..max_new fresh nodes wired to the same outside producers and consumers."""
    op, shp, es, ed = g["op"], g["shape"], g["edge_src"], g["edge_dst"]
    n, S = shp.shape
    length = int(rng.integers(2, max_region + 1))
    r = int(rng.integers(1, max_new + 1))
    s = int(rng.integers(1, max(2, n - length)))
    e = min(n, s + length)
    shift = r - (e - s)

    src_in = (es >= s) & (es < e)
    dst_in = (ed >= s) & (ed < e)
    keep = ~dst_in & ~(src_in & dst_in)
    producers = np.unique(es[dst_in & ~src_in])

    new_src = es[keep].copy()
    new_dst = ed[keep].copy()
    rewired = src_in[keep]                       # region -> outside consumer
    new_src[rewired] = s + rng.integers(0, r, size=int(rewired.sum()))
    new_src[~rewired & (new_src >= e)] += shift
    new_dst[new_dst >= e] += shift

    add_s, add_d = [], []
    for k in range(r):
        pool = np.concatenate([producers, np.arange(s, s + k)])
        if len(pool) == 0:
            continue
        deg = int(rng.integers(1, min(3, len(pool)) + 1))
        for p in rng.choice(pool, size=deg, replace=False):
            add_s.append(int(p)); add_d.append(s + k)

    # which node of the original each node of the candidate is (-1 for the fresh ones)
    twin = np.concatenate([np.arange(s), np.full(r, -1), np.arange(e, n)]).astype(np.int32)
    return {
        "twin": twin,
        "op": np.concatenate([op[:s], rng.integers(0, T, size=r).astype(np.int32), op[e:]]),
        "shape": np.concatenate([shp[:s], shape_features(rng, r, S, bf16), shp[e:]]),
        "edge_src": np.concatenate([new_src, np.asarray(add_s, dtype=np.int32)]).astype(np.int32),
        "edge_dst": np.concatenate([new_dst, np.asarray(add_d, dtype=np.int32)]).astype(np.int32),
    }


def tensor_shape_attributes(rng, num_edges, S=8, bf16=False, M=4096.0):
    """Per-edge attributes as the paper describes them (Section 3.3.2): the shape of the tensor an edge
    carries as four dimensions divided by the constant M, ranks below four padded with zeros in the leading
    positions; the remaining S - 4 columns are zero.  Input data only (no arithmetic of the method)."""
    a = np.zeros((num_edges, S), dtype=np.float32)
    rank = rng.integers(1, 5, size=num_edges)
    dims = np.exp2(rng.uniform(0.0, 12.0, size=(num_edges, 4))).astype(np.int64).clip(1, 4096)
    for r in range(1, 5):
        rows = rank == r
        a[rows, 4 - r:4] = dims[rows, 4 - r:4] / M
    return round_to_bf16_grid(a) if bf16 else a


def flatten(graphs, env_off, A_max, mask=None):
    """Concatenate per-graph arrays into the flat batch both sides consume."""
    env_off = np.asarray(env_off, dtype=np.int32)
    num_envs = len(env_off) - 1
    if mask is None:
        mask = np.zeros((num_envs, A_max), dtype=np.uint8)
        for e in range(num_envs):
            mask[e, : env_off[e + 1] - env_off[e] - 1] = 1
    S = graphs[0]["shape"].shape[1]
    # base_id: packed id of the current-graph node a candidate node was copied from (-1: none)
    node_off = np.concatenate([[0], np.cumsum([len(g["op"]) for g in graphs])])
    base_id = np.full(int(node_off[-1]), -1, dtype=np.int32)
    for e in range(num_envs):
        cur = int(env_off[e])
        for gi in range(cur + 1, int(env_off[e + 1])):
            tw = graphs[gi].get("twin")
            if tw is not None:
                base_id[node_off[gi]:node_off[gi + 1]] = np.where(tw >= 0, tw + node_off[cur], -1)
    extra = {}
    if len(graphs) and all(g.get("edge_attr") is not None for g in graphs):      # attributes on the edges
        extra["edge_attr"] = np.ascontiguousarray(
            np.concatenate([np.asarray(g["edge_attr"], dtype=np.float32).reshape(-1, S) for g in graphs]))
    return {
        **extra,
        "base_id": base_id,
        "num_graphs": len(graphs),
        "n_nodes": np.array([len(g["op"]) for g in graphs], dtype=np.int32),
        "n_edges": np.array([len(g["edge_src"]) for g in graphs], dtype=np.int32),
        "op": np.ascontiguousarray(np.concatenate([g["op"] for g in graphs]), dtype=np.int32),
        "shape": np.ascontiguousarray(
            np.concatenate([g["shape"].reshape(-1, S) for g in graphs]), dtype=np.float32),
        "edge_src": np.ascontiguousarray(
            np.concatenate([g["edge_src"] for g in graphs]), dtype=np.int32),
        "edge_dst": np.ascontiguousarray(
            np.concatenate([g["edge_dst"] for g in graphs]), dtype=np.int32),
        "env_off": env_off,
        "mask": np.ascontiguousarray(mask, dtype=np.uint8),
    }


def split(batch):
    """Inverse of flatten(): the list of per-graph dicts (views into the flat arrays)."""
    no = np.concatenate([[0], np.cumsum(batch["n_nodes"])])
    eo = np.concatenate([[0], np.cumsum(batch["n_edges"])])
    return [{
        "op": batch["op"][no[g]:no[g + 1]],
        "shape": batch["shape"][no[g]:no[g + 1]],
        "edge_src": batch["edge_src"][eo[g]:eo[g + 1]],
        "edge_dst": batch["edge_dst"][eo[g]:eo[g + 1]],
    } for g in range(batch["num_graphs"])]

"""Dense-adjacency restatement of the encoder in numpy, used to pin the oracle.

Written independently of oracle/: the graph is an n x n multiplicity matrix and every
step is a dense matrix expression, so an indexing slip in the oracle's CSR walk or a
dropped term shows up as a mismatch on tiny graphs.
"""
import numpy as np


def bf16_round(x):
    x = np.asarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def adjacency(g):
    n = len(g["op"])
    A = np.zeros((n, n))
    for s, d in zip(g["edge_src"], g["edge_dst"]):
        A[d, s] += 1.0          # row = consumer, column = producer
    return A


def node_update(g, W, m):
    """Eq. 6 as X @ W0 + b0 with X = [A @ shape || onehot(op) || shape]; with attributes on the edges
    (g["edge_attr"], one row per edge of the input list) the first block is the incidence matrix (consumer
    x edge) times the attributes instead."""
    A = adjacency(g)
    # a bf16 model stores its input features in bf16: arbitrary reals are rounded once, up front
    as_stored = bf16_round if m["dtype"] == "bf16" else (lambda a: np.asarray(a, dtype=np.float64))
    shp = as_stored(g["shape"])
    onehot = np.eye(m["T"])[g["op"]]
    if g.get("edge_attr") is not None:
        n, ne = len(g["op"]), len(g["edge_dst"])
        Inc = np.zeros((n, ne))
        Inc[np.asarray(g["edge_dst"]), np.arange(ne)] = 1.0
        agg = Inc @ as_stored(g["edge_attr"])
    else:
        agg = A @ shp
    X = np.concatenate([agg, onehot, shp], axis=1)
    W0 = bf16_round(W["W0"]) if m["dtype"] == "bf16" else W["W0"].astype(np.float64)
    return np.maximum(X @ W0 + W["b0"].astype(np.float64), 0.0)


def gat_layer(g, h, W, l, m, return_alpha=False):
    """Eq. 7 with the multiplicity matrix M = A + I weighting a dense row softmax."""
    n = len(g["op"])
    K, H = m["K"], m["H"]
    d = H // K
    Wl = W[f"W{l}"]
    Wl = bf16_round(Wl) if m["dtype"] == "bf16" else Wl.astype(np.float64)
    Z = h @ Wl
    A = adjacency(g)
    M = A + np.eye(n) + (A.T if m.get("both_ways") else 0.0)     # consumers count as neighbours too
    out = np.zeros((n, H))
    alphas = []
    for k in range(K):
        Zk = Z[:, k * d:(k + 1) * d]
        s_src = Zk @ W[f"a_src{l}"][k * d:(k + 1) * d].astype(np.float64)
        s_dst = Zk @ W[f"a_dst{l}"][k * d:(k + 1) * d].astype(np.float64)
        e = s_dst[:, None] + s_src[None, :]
        e = np.where(e > 0, e, 0.2 * e)
        e = np.where(M > 0, e, -np.inf)
        p = M * np.exp(e - e.max(axis=1, keepdims=True))
        alpha = p / p.sum(axis=1, keepdims=True)
        alphas.append(alpha)
        out[:, k * d:(k + 1) * d] = alpha @ Zk
    out = np.maximum(out + W[f"b{l}"].astype(np.float64), 0.0)
    return (out, alphas) if return_alpha else out


def global_update(h, W, m, g_attr=None):
    """Eq. 8: ReLU(Wg^T [sum_i h_i || g] + bg)."""
    ga = np.zeros(m["Dg"]) if g_attr is None else np.asarray(g_attr, dtype=np.float64)
    u = np.concatenate([h.sum(axis=0), ga])
    return np.maximum(u @ W["Wg"].astype(np.float64) + W["bg"].astype(np.float64), 0.0)


def encode_graph(g, W, m, g_attr=None):
    h = node_update(g, W, m)
    for l in range(1, m["L"] + 1):
        h = gat_layer(g, h, W, l, m)
    return global_update(h, W, m, g_attr)


def mlp(x, W1, b1, w2, b2, Wh=None, bh=None):
    y = np.maximum(x @ W1.astype(np.float64) + b1, 0.0)
    if Wh is not None:                      # second hidden layer
        y = np.maximum(y @ Wh.astype(np.float64) + bh, 0.0)
    return float(y @ w2.astype(np.float64) + b2[0])

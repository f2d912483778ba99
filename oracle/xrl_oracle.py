"""ctypes front end of the CPU oracle (test infrastructure; see xrl_oracle.cpp).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_lib = None

_i32p = C.POINTER(C.c_int32)
_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)
_u8p = C.POINTER(C.c_uint8)


class _Model(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("T", "S", "H", "K", "L", "Hm", "Dg", "dtype", "Hm2", "nbr")]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.xo_philox4x32_10.restype = None
        _lib.xo_philox4x32_10.argtypes = [C.c_uint32] * 6 + [C.POINTER(C.c_uint32)]
        _lib.xo_sample.argtypes = [C.c_int32, C.c_int32, _f32p, C.c_uint64, C.c_uint64, _i32p]
    return _lib


def _p(a, t):
    return None if a is None else a.ctypes.data_as(t)


def _model(m):
    return _Model(m["T"], m["S"], m["H"], m["K"], m["L"], m["Hm"], m["Dg"],
                  1 if m["dtype"] == "bf16" else 0, int(m.get("Hm2", 0)), 1 if m.get("both_ways") else 0)


def num_threads():
    return int(lib().xo_num_threads())


def philox4x32_10(key, counter):
    out = (C.c_uint32 * 4)()
    lib().xo_philox4x32_10(key[0], key[1], counter[0], counter[1], counter[2], counter[3], out)
    return [int(v) for v in out]


def pack(batch):
    """Section 3.3.2 meta-graph.  Returns (status, dict of int32 arrays)."""
    B = int(batch["num_graphs"])
    N = int(batch["n_nodes"].sum()); E = int(batch["n_edges"].sum())
    env_off = np.ascontiguousarray(batch["env_off"], dtype=np.int32)
    out = {
        "node_off": np.zeros(B + 1, np.int32), "edge_off": np.zeros(B + 1, np.int32),
        "seg_id": np.zeros(N, np.int32), "graph_env": np.zeros(B, np.int32),
        "rowptr": np.zeros(N + 1, np.int32), "col": np.zeros(E, np.int32),
        "eid": np.zeros(E, np.int32),
    }
    st = lib().xo_pack(
        C.c_int32(B), _p(batch["n_nodes"], _i32p), _p(batch["n_edges"], _i32p),
        _p(batch["edge_src"], _i32p), _p(batch["edge_dst"], _i32p),
        C.c_int32(len(env_off) - 1), _p(env_off, _i32p),
        _p(out["node_off"], _i32p), _p(out["edge_off"], _i32p), _p(out["seg_id"], _i32p),
        _p(out["graph_env"], _i32p), _p(out["rowptr"], _i32p), _p(out["col"], _i32p),
        _p(out["eid"], _i32p))
    return int(st), out


def encode(m, weights, batch, packed, g0=None, sel=None, mode=0, threads=0, dump_layer=-1,
           want_nodes=False, want_alpha=False, edge_attr=None):
    """Section 3.4 (Eq. 6, Eq. 7 x L, Eq. 8).  Returns dict(emb[, nodes, alpha_edge, alpha_self]).
    edge_attr ([E x S] float32, input edge order; default batch.get("edge_attr")): attributes on edges in
    Eq. 6 instead of the producers' shape features."""
    if edge_attr is None:
        edge_attr = batch.get("edge_attr")
    ea = None if edge_attr is None else np.ascontiguousarray(edge_attr, dtype=np.float32)
    B = int(batch["num_graphs"])
    N = int(batch["n_nodes"].sum()); E = int(batch["n_edges"].sum())
    weights = np.ascontiguousarray(weights, dtype=np.float32)
    shape = np.ascontiguousarray(batch["shape"], dtype=np.float32)
    op = np.ascontiguousarray(batch["op"], dtype=np.int32)
    sel_a = None if sel is None else np.ascontiguousarray(sel, dtype=np.int32)
    n_out = B if sel is None else len(sel_a)
    emb = np.zeros((n_out, m["H"]), np.float64)
    nodes = np.full((N, m["H"]), np.nan, np.float64) if want_nodes else None
    a_e = np.full((E, m["K"]), np.nan, np.float64) if want_alpha else None
    a_s = np.full((N, m["K"]), np.nan, np.float64) if want_alpha else None
    g0a = None if g0 is None else np.ascontiguousarray(g0, dtype=np.float64)
    mm = _model(m)
    st = lib().xo_encode(
        C.byref(mm), _p(weights, _f32p), C.c_int32(B), _p(packed["node_off"], _i32p),
        _p(packed["rowptr"], _i32p), _p(packed["col"], _i32p), _p(op, _i32p), _p(shape, _f32p),
        _p(g0a, _f64p), C.c_int32(n_out), _p(sel_a, _i32p), C.c_int32(mode), C.c_int32(threads),
        _p(emb, _f64p), C.c_int32(dump_layer), _p(nodes, _f64p), _p(a_e, _f64p), _p(a_s, _f64p),
        _p(ea, _f32p), _p(packed["eid"] if ea is not None else None, _i32p))
    if st != 0:
        raise ValueError(f"xo_encode status {st}")
    return {"emb": emb, "nodes": nodes, "alpha_edge": a_e, "alpha_self": a_s}


def policy_value(m, weights, batch, emb, mask=None):
    """Sections 3.3.2 / 3.3.3 heads.  Returns (status, logits, probs, value)."""
    env_off = np.ascontiguousarray(batch["env_off"], dtype=np.int32)
    Ne = len(env_off) - 1
    A = int(m["A_max"])
    mask = np.ascontiguousarray(batch["mask"] if mask is None else mask, dtype=np.uint8)
    weights = np.ascontiguousarray(weights, dtype=np.float32)
    emb = np.ascontiguousarray(emb, dtype=np.float64)
    logits = np.zeros((Ne, A + 1)); probs = np.zeros((Ne, A + 1)); value = np.zeros(Ne)
    mm = _model(m)
    st = lib().xo_policy_value(C.byref(mm), _p(weights, _f32p), C.c_int32(Ne), _p(env_off, _i32p),
                               C.c_int32(A), _p(emb, _f64p), _p(mask, _u8p), _p(logits, _f64p),
                               _p(probs, _f64p), _p(value, _f64p))
    return int(st), logits, probs, value


def sample(probs_f32, seed, step):
    """Integer-CDF categorical draw per environment from fp32 probabilities."""
    p = np.ascontiguousarray(probs_f32, dtype=np.float32)
    Ne, A1 = p.shape
    act = np.zeros(Ne, np.int32)
    st = lib().xo_sample(C.c_int32(Ne), C.c_int32(A1), _p(p, _f32p), C.c_uint64(seed),
                         C.c_uint64(step), _p(act, _i32p))
    if st != 0:
        raise ValueError(f"xo_sample status {st}")
    return act


def init_weights(m, seed):
    """The seeded Xavier-uniform weight blob the library's xrl_init_weights defines (float32)."""
    from workloads import configs
    n = configs.weight_count(m)
    out = np.zeros(n, np.float32)
    fn = lib().xo_init_weights
    fn.restype = C.c_int64
    mm = _model(m)
    wrote = fn(C.byref(mm), C.c_uint64(int(seed)), _p(out, _f32p))
    if wrote != n:
        raise ValueError(f"xo_init_weights wrote {wrote} of {n}")
    return out


def forward(m, weights, batch, g0=None, threads=0, mode=0):
    """Whole step: pack -> encode -> heads.  Convenience for tests and the CPU baseline."""
    st, packed = pack(batch)
    if st != 0:
        raise ValueError(f"xo_pack status {st}")
    enc = encode(m, weights, batch, packed, g0=g0, threads=threads, mode=mode)
    st, logits, probs, value = policy_value(m, weights, batch, enc["emb"])
    if st != 0:
        raise ValueError(f"xo_policy_value status {st}")
    return {"packed": packed, "emb": enc["emb"], "logits": logits, "probs": probs, "value": value}


def ppo_grad(m, weights, batch, packed, action, logp_old, adv, ret, eps=0.2, c1=0.5, c2=0.01, g0=None,
             mask=None, edge_attr=None, mirrored=False):
    """Section 3.3.4, Eq. 3-5 over the environments of the batch (each a stored transition) and the gradient
    of J with respect to the weight blob.  Returns dict(loss=[J, L_clip, L_vf, L_ent], grad (float64, blob
    shaped), logp [num_envs]).  mirrored: keep Z and the layer outputs as a bf16 model stores them (debugging
    aid; the definition is mirrored=False); mirrored=2 also takes the half-scores from the rounded Z."""
    B = int(batch["num_graphs"])
    weights = np.ascontiguousarray(weights, dtype=np.float32)
    shape = np.ascontiguousarray(batch["shape"], dtype=np.float32)
    op = np.ascontiguousarray(batch["op"], dtype=np.int32)
    env_off = np.ascontiguousarray(batch["env_off"], dtype=np.int32)
    Ne = len(env_off) - 1
    A = int(m["A_max"])
    mask = np.ascontiguousarray(batch["mask"] if mask is None else mask, dtype=np.uint8)
    if edge_attr is None:
        edge_attr = batch.get("edge_attr")
    ea = None if edge_attr is None else np.ascontiguousarray(edge_attr, dtype=np.float32)
    g0a = None if g0 is None else np.ascontiguousarray(g0, dtype=np.float64)
    action = np.ascontiguousarray(action, dtype=np.int32)
    logp_old = np.ascontiguousarray(logp_old, dtype=np.float64)
    adv = np.ascontiguousarray(adv, dtype=np.float64)
    ret = np.ascontiguousarray(ret, dtype=np.float64)
    loss = np.zeros(4)
    grad = np.zeros(len(weights))
    logp = np.zeros(Ne)
    mm = _model(m)
    st = lib().xo_ppo_grad(
        C.byref(mm), _p(weights, _f32p), C.c_int32(B), _p(packed["node_off"], _i32p),
        _p(packed["rowptr"], _i32p), _p(packed["col"], _i32p), _p(op, _i32p), _p(shape, _f32p),
        _p(g0a, _f64p), _p(ea, _f32p), _p(packed["eid"] if ea is not None else None, _i32p),
        C.c_int32(Ne), _p(env_off, _i32p), C.c_int32(A), _p(mask, _u8p), _p(action, _i32p),
        _p(logp_old, _f64p), _p(adv, _f64p), _p(ret, _f64p), C.c_double(eps), C.c_double(c1),
        C.c_double(c2), _p(loss, _f64p), _p(grad, _f64p), _p(logp, _f64p), C.c_int32(int(mirrored)))
    if st != 0:
        raise ValueError(f"xo_ppo_grad status {st}")
    return {"loss": loss, "grad": grad, "logp": logp}


def gae(reward, values, done, gamma, lam):
    """Generalised advantage estimates of one trajectory: values has len(reward) + 1 entries.  Returns
    (advantages, value targets)."""
    reward = np.ascontiguousarray(reward, dtype=np.float64)
    values = np.ascontiguousarray(values, dtype=np.float64)
    done = np.ascontiguousarray(done, dtype=np.uint8)
    T = len(reward)
    assert len(values) == T + 1 and len(done) == T
    adv = np.zeros(T); ret = np.zeros(T)
    st = lib().xo_gae(C.c_int32(T), _p(reward, _f64p), _p(values, _f64p), _p(done, _u8p),
                      C.c_double(gamma), C.c_double(lam), _p(adv, _f64p), _p(ret, _f64p))
    if st != 0:
        raise ValueError(f"xo_gae status {st}")
    return adv, ret

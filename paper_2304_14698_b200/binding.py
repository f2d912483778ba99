"""ctypes binding of libxrl.so: one Python function per C entry point, same names.

Only argument marshalling happens here.  Device buffers are torch CUDA tensors (torch is used
for device memory and streams, nothing else); every function takes raw pointers from them.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libxrl.so")
_lib = None

STATUS_NAMES = {0: "XRL_OK", 1: "XRL_ERR_INVALID_ARG", 2: "XRL_ERR_BAD_GRAPH", 3: "XRL_ERR_CAPACITY",
                4: "XRL_ERR_ALLOC", 5: "XRL_ERR_CUDA", 6: "XRL_ERR_STATE", 7: "XRL_ERR_TIMEOUT",
                8: "XRL_ERR_UNSUPPORTED"}
XRL_FP32, XRL_BF16 = 0, 1
XRL_MEM_HOST, XRL_MEM_DEVICE = 0, 1

EXPORTED_SYMBOLS = [
    "xrl_create", "xrl_destroy", "xrl_weights_size", "xrl_set_weights", "xrl_pack", "xrl_pack_flat",
    "xrl_batch_free", "xrl_batch_info", "xrl_batch_export", "xrl_encode", "xrl_debug_node_features",
    "xrl_policy_value", "xrl_sample", "xrl_last_device_status", "xrl_launch_counts", "xrl_version",
    "xrl_profile", "xrl_profile_read", "xrl_pack_csr_static", "xrl_encode_delta", "xrl_delta_rows", "xrl_get_weights",
    "xrl_graph_begin", "xrl_graph_launch", "xrl_batch_set_edge_attr", "xrl_ppo_grad", "xrl_gae",
    "xrl_grad_weigh", "xrl_grad_unweigh", "xrl_init_weights",
]
PROFILE_FAMILIES = ["pack", "node_update", "transform", "aggregate", "readout", "heads", "aggregate_readout",
                    "layers_fused"]


class XrlError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__(f"{where}: {STATUS_NAMES.get(int(status), status)}")


class _ModelConfig(C.Structure):
    _fields_ = [("num_op_types", C.c_int32), ("num_shape_feats", C.c_int32), ("hidden", C.c_int32),
                ("heads", C.c_int32), ("layers", C.c_int32), ("mlp_hidden", C.c_int32),
                ("mlp_hidden2", C.c_int32), ("global_dim", C.c_int32), ("dtype", C.c_int32),
                ("edge_attributes", C.c_int32), ("neighbourhood", C.c_int32), ("max_actions", C.c_int32),
                ("max_graphs", C.c_int32), ("max_envs", C.c_int32), ("max_nodes", C.c_int64),
                ("max_edges", C.c_int64)]


class _Graph(C.Structure):
    _fields_ = [("num_nodes", C.c_int32), ("num_edges", C.c_int32), ("op", C.c_void_p),
                ("shape", C.c_void_p), ("edge_src", C.c_void_p), ("edge_dst", C.c_void_p)]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libxrl.so.  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with "
                          "`python -m paper_2304_14698_b200.build` (needs nvcc)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    sigs = {
        "xrl_create": [C.POINTER(_ModelConfig), i32, C.POINTER(vp)],
        "xrl_destroy": [vp],
        "xrl_weights_size": [vp, C.POINTER(C.c_size_t)],
        "xrl_set_weights": [vp, vp, C.c_size_t],
        "xrl_get_weights": [vp, vp, C.c_size_t],
        "xrl_init_weights": [vp, u64],
        "xrl_pack": [vp, C.POINTER(_Graph), i32, vp, i32, vp, C.POINTER(vp)],
        "xrl_pack_flat": [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, i32, vp, C.POINTER(vp)],
        "xrl_batch_free": [vp, vp],
        "xrl_batch_info": [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i32), C.POINTER(i32)],
        "xrl_batch_export": [vp, vp, vp, vp, vp, vp, vp],
        "xrl_encode": [vp, vp, vp, vp, vp],
        "xrl_debug_node_features": [vp, vp, i32, vp, vp],
        "xrl_policy_value": [vp, vp, vp, vp, vp, vp, vp, u64, u64, vp],
        "xrl_sample": [vp, vp, i32, i32, u64, u64, vp, vp],
        "xrl_last_device_status": [vp, vp, C.POINTER(i32)],
        "xrl_launch_counts": [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)],
        "xrl_profile": [vp, i32],
        "xrl_encode_delta": [vp, vp, vp, vp, vp, vp],
        "xrl_delta_rows": [vp, C.POINTER(i64), i32],
        "xrl_pack_csr_static": [i32, i32, i32] + [vp] * 6 + [i32] + [vp] * 8,
        "xrl_profile_read": [vp, C.POINTER(C.c_double), C.POINTER(i64), i32],
        "xrl_batch_set_edge_attr": [vp, vp, i32, vp, vp],
        "xrl_graph_begin": [vp],
        "xrl_ppo_grad": [vp] * 8 + [C.c_float] * 3 + [vp] * 4,
        "xrl_gae": [i32, i32, i32, vp, vp, vp, C.c_float, C.c_float, vp, vp, vp],
        "xrl_graph_launch": [vp, vp],
        "xrl_grad_weigh": [i32, i32, i32, vp, i64, vp, i64, vp, vp],
        "xrl_grad_unweigh": [i32, i32, i32, vp, i64, vp, vp, C.POINTER(i64), vp],
    }
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = None if name == "xrl_destroy" else C.c_int32
    lib.xrl_version.restype = C.c_char_p
    lib.xrl_version.argtypes = []
    _lib = lib
    return lib


def _check(st, where):
    if st != 0:
        raise XrlError(st, where)


def _np_ptr(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _dev_ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(int(stream))


def model_config(m, max_graphs, max_envs, max_nodes, max_edges):
    """Build the C config from a dict with keys T, S, H, K, L, Hm, Dg, dtype, A_max and, optionally,
    Hm2 (second hidden width of the heads' MLPs, default 0 = one hidden layer) and edge_attr (True: the
    model takes Eq. 6's edge attributes from the edges themselves, see xrl_batch_set_edge_attr) and
    both_ways (True: Eq. 7's neighbours of a node are its producers and its consumers)."""
    return _ModelConfig(m["T"], m["S"], m["H"], m["K"], m["L"], m["Hm"], int(m.get("Hm2", 0)), m["Dg"],
                        XRL_BF16 if m["dtype"] in ("bf16", XRL_BF16) else XRL_FP32,
                        1 if m.get("edge_attr") else 0, 1 if m.get("both_ways") else 0, m["A_max"],
                        int(max_graphs), int(max_envs), int(max_nodes), int(max_edges))


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16).reshape(x.shape)


# ---- one function per C entry point ---------------------------------------------------------

def xrl_version() -> str:
    return load_library().xrl_version().decode()


def xrl_create(cfg: _ModelConfig, device: int = 0):
    out = C.c_void_p()
    _check(load_library().xrl_create(C.byref(cfg), device, C.byref(out)), "xrl_create")
    return out


def xrl_destroy(ctx):
    load_library().xrl_destroy(ctx)


def xrl_weights_size(ctx) -> int:
    n = C.c_size_t()
    _check(load_library().xrl_weights_size(ctx, C.byref(n)), "xrl_weights_size")
    return int(n.value)


def xrl_set_weights(ctx, blob: np.ndarray):
    blob = np.ascontiguousarray(blob, dtype=np.float32)
    _check(load_library().xrl_set_weights(ctx, _np_ptr(blob), blob.nbytes), "xrl_set_weights")


def xrl_init_weights(ctx, seed: int):
    """Seeded Xavier-uniform weights (see include/xrl.h) in place of xrl_set_weights."""
    _check(load_library().xrl_init_weights(ctx, int(seed)), "xrl_init_weights")


def xrl_get_weights(ctx) -> np.ndarray:
    blob = np.zeros(xrl_weights_size(ctx) // 4, np.float32)
    _check(load_library().xrl_get_weights(ctx, _np_ptr(blob), blob.nbytes), "xrl_get_weights")
    return blob


def xrl_pack(ctx, graphs, env_off, dtype, stream=None, batch=None):
    """graphs: list of dicts (op int32[n], shape float32[n,S], edge_src, edge_dst) in HOST memory."""
    keep = []
    arr = (_Graph * max(1, len(graphs)))()
    for i, g in enumerate(graphs):
        op = np.ascontiguousarray(g["op"], dtype=np.int32)
        shp = np.ascontiguousarray(g["shape"], dtype=np.float32)
        if dtype in ("bf16", XRL_BF16):
            shp = to_bf16_bits(shp)
        es = np.ascontiguousarray(g["edge_src"], dtype=np.int32)
        ed = np.ascontiguousarray(g["edge_dst"], dtype=np.int32)
        keep += [op, shp, es, ed]
        arr[i] = _Graph(len(op), len(es), op.ctypes.data, shp.ctypes.data, es.ctypes.data, ed.ctypes.data)
    env_off = np.ascontiguousarray(env_off, dtype=np.int32)
    out = C.c_void_p(batch.value if batch is not None else None)
    st = load_library().xrl_pack(ctx, arr, len(graphs), _np_ptr(env_off), len(env_off) - 1,
                                 _stream(stream), C.byref(out))
    _check(st, "xrl_pack")
    return out


def xrl_pack_flat(ctx, where, n_nodes, n_edges, op, shape, edge_src, edge_dst, env_off, stream=None,
                  batch=None):
    """Counts and env_off: numpy int32 (HOST).  Bulk arrays: numpy (where = HOST) or torch CUDA
    tensors (where = DEVICE); shape must already have the storage type (float32 or bf16)."""
    n_nodes = np.ascontiguousarray(n_nodes, dtype=np.int32)
    n_edges = np.ascontiguousarray(n_edges, dtype=np.int32)
    env_off = np.ascontiguousarray(env_off, dtype=np.int32)
    ptr = _np_ptr if where == XRL_MEM_HOST else _dev_ptr
    out = C.c_void_p(batch.value if batch is not None else None)
    st = load_library().xrl_pack_flat(ctx, where, len(n_nodes), _np_ptr(n_nodes), _np_ptr(n_edges),
                                      ptr(op), ptr(shape), ptr(edge_src), ptr(edge_dst),
                                      _np_ptr(env_off), len(env_off) - 1, _stream(stream), C.byref(out))
    _check(st, "xrl_pack_flat")
    return out


def xrl_batch_set_edge_attr(ctx, batch, edge_attr, stream=None):
    """edge_attr: [E, S] in the storage type, rows in the order of the packed edge lists; numpy (HOST;
    float32, or uint16 bf16 bits) or a torch CUDA tensor (DEVICE)."""
    on_dev = not isinstance(edge_attr, np.ndarray)
    ptr = _dev_ptr(edge_attr) if on_dev else _np_ptr(np.ascontiguousarray(edge_attr))
    _check(load_library().xrl_batch_set_edge_attr(ctx, batch, XRL_MEM_DEVICE if on_dev else XRL_MEM_HOST, ptr,
                                                  _stream(stream)), "xrl_batch_set_edge_attr")


def xrl_batch_free(ctx, batch):
    _check(load_library().xrl_batch_free(ctx, batch), "xrl_batch_free")


def xrl_batch_info(batch):
    n, e, b, ne = C.c_int64(), C.c_int64(), C.c_int32(), C.c_int32()
    _check(load_library().xrl_batch_info(batch, C.byref(n), C.byref(e), C.byref(b), C.byref(ne)),
           "xrl_batch_info")
    return {"num_nodes": n.value, "num_edges": e.value, "num_graphs": b.value, "num_envs": ne.value}


def xrl_batch_export(batch):
    info = xrl_batch_info(batch)
    N, E, B = info["num_nodes"], info["num_edges"], info["num_graphs"]
    out = {"rowptr": np.zeros(N + 1, np.int32), "col": np.zeros(E, np.int32),
           "seg_id": np.zeros(N, np.int32), "node_off": np.zeros(B + 1, np.int32),
           "edge_off": np.zeros(B + 1, np.int32), "graph_env": np.zeros(B, np.int32)}
    st = load_library().xrl_batch_export(batch, _np_ptr(out["rowptr"]), _np_ptr(out["col"]),
                                         _np_ptr(out["seg_id"]), _np_ptr(out["node_off"]),
                                         _np_ptr(out["edge_off"]), _np_ptr(out["graph_env"]))
    _check(st, "xrl_batch_export")
    return out


def xrl_encode(ctx, batch, graph_emb, g0=None, stream=None):
    """graph_emb: torch CUDA float32 [B, H] (written).  g0: torch CUDA float32 [B, Dg] or None."""
    _check(load_library().xrl_encode(ctx, batch, _dev_ptr(g0), _dev_ptr(graph_emb), _stream(stream)),
           "xrl_encode")
    return graph_emb


def xrl_encode_delta(ctx, batch, base_id, graph_emb, g0=None, stream=None):
    """Like xrl_encode, recomputing only what a candidate's rewrite can change.  base_id: torch CUDA int32
    [N] hint (packed id of the equal node of the env's current graph, or -1), or None."""
    _check(load_library().xrl_encode_delta(ctx, batch, _dev_ptr(base_id), _dev_ptr(g0), _dev_ptr(graph_emb),
                                           _stream(stream)), "xrl_encode_delta")
    return graph_emb


def xrl_delta_rows(ctx, layers):
    rows = (C.c_int64 * (layers + 1))()
    _check(load_library().xrl_delta_rows(ctx, rows, layers + 1), "xrl_delta_rows")
    return [int(v) for v in rows]


def xrl_debug_node_features(ctx, batch, num_layers, hidden, stream=None):
    info = xrl_batch_info(batch)
    out = np.zeros((info["num_nodes"], hidden), np.float32)
    _check(load_library().xrl_debug_node_features(ctx, batch, num_layers, _np_ptr(out), _stream(stream)),
           "xrl_debug_node_features")
    return out


def xrl_policy_value(ctx, batch, graph_emb, mask, probs, value, action=None, seed=0, step=0,
                     stream=None):
    st = load_library().xrl_policy_value(ctx, batch, _dev_ptr(graph_emb), _dev_ptr(mask), _dev_ptr(probs),
                                         _dev_ptr(value), _dev_ptr(action), seed, step, _stream(stream))
    _check(st, "xrl_policy_value")
    return probs, value, action


def xrl_sample(ctx, probs, action, seed, step, stream=None):
    ne, a1 = probs.shape
    _check(load_library().xrl_sample(ctx, _dev_ptr(probs), ne, a1, seed, step, _dev_ptr(action),
                                     _stream(stream)), "xrl_sample")
    return action


def xrl_ppo_grad(ctx, batch, mask, action, logp_old, adv, ret, loss_out, grad, eps=0.2, c1=0.5, c2=0.01,
                 g0=None, logp_out=None, stream=None):
    """Section 3.3.4: loss_out[4] = {J, L_clip, L_vf, L_ent} and grad (blob-shaped fp32), all device tensors."""
    st = load_library().xrl_ppo_grad(ctx, batch, _dev_ptr(g0), _dev_ptr(mask), _dev_ptr(action),
                                     _dev_ptr(logp_old), _dev_ptr(adv), _dev_ptr(ret), C.c_float(eps),
                                     C.c_float(c1), C.c_float(c2), _dev_ptr(loss_out), _dev_ptr(grad),
                                     _dev_ptr(logp_out), _stream(stream))
    _check(st, "xrl_ppo_grad")
    return loss_out, grad


def xrl_gae(reward, values, done, gamma, lam, adv=None, ret=None, stream=None):
    """Generalised advantage estimates of M trajectories, step-major device tensors: reward, done [T x M],
    values [(T + 1) x M] -> (adv, ret) [T x M]."""
    import torch
    T, M = reward.shape
    adv = torch.empty_like(reward) if adv is None else adv
    ret = torch.empty_like(reward) if ret is None else ret
    st = load_library().xrl_gae(reward.device.index or 0, T, M, _dev_ptr(reward), _dev_ptr(values), _dev_ptr(done),
                                C.c_float(gamma), C.c_float(lam), _dev_ptr(adv), _dev_ptr(ret), _stream(stream))
    _check(st, "xrl_gae")
    return adv, ret


def _where_ptr(t):
    """(where, device index, pointer) of a contiguous torch tensor that lives on the CPU or on a CUDA device."""
    if t.is_cuda:
        return XRL_MEM_DEVICE, t.device.index or 0, C.c_void_p(t.data_ptr())
    return XRL_MEM_HOST, 0, C.c_void_p(t.data_ptr())


def xrl_grad_weigh(grad, loss, num_envs, buf, stream=None):
    """buf[count + 5] = [grad * n | loss * n | n] (see include/xrl.h); torch tensors, all on one device or all on
    the CPU, float32 or float64."""
    where, dev, gp = _where_ptr(grad)
    st = _stream(stream) if where == XRL_MEM_DEVICE else None
    _check(load_library().xrl_grad_weigh(where, dev, grad.element_size(), gp, grad.numel(), _where_ptr(loss)[2],
                                         int(num_envs), _where_ptr(buf)[2], st), "xrl_grad_weigh")
    return buf


def xrl_grad_unweigh(buf, grad, loss, stream=None) -> int:
    """grad, loss = buf / buf[-1]; returns the total number of environments (synchronises for device buffers)."""
    where, dev, gp = _where_ptr(grad)
    st = _stream(stream) if where == XRL_MEM_DEVICE else None
    total = C.c_int64()
    _check(load_library().xrl_grad_unweigh(where, dev, grad.element_size(), _where_ptr(buf)[2], grad.numel(), gp,
                                           _where_ptr(loss)[2], C.byref(total), st), "xrl_grad_unweigh")
    return int(total.value)


def allreduce_ppo_grad(loss, grad, num_envs, group=None):
    """Data-parallel training step: every rank has run xrl_ppo_grad on its own environments, so its loss terms
    and gradient are means over `num_envs` local environments.  In place, they become the means over all
    ranks' environments: xrl_grad_weigh, one sum all-reduce of the buffer (NCCL for device tensors),
    xrl_grad_unweigh.  The result equals one xrl_ppo_grad call on the concatenated batch.  loss [4] and grad are
    contiguous torch tensors of one floating type on one device.  Returns the global number of environments."""
    import torch
    import torch.distributed as dist
    buf = torch.empty(grad.numel() + 5, dtype=grad.dtype, device=grad.device)
    xrl_grad_weigh(grad, loss, num_envs, buf)
    dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
    return xrl_grad_unweigh(buf, grad, loss)


def xrl_last_device_status(ctx, stream=None) -> int:
    s = C.c_int32()
    _check(load_library().xrl_last_device_status(ctx, _stream(stream), C.byref(s)),
           "xrl_last_device_status")
    return int(s.value)


def xrl_graph_begin(ctx):
    """Start recording the kernels of the following xrl_encode / xrl_policy_value / xrl_sample calls."""
    _check(load_library().xrl_graph_begin(ctx), "xrl_graph_begin")


def xrl_graph_launch(ctx, stream=None):
    """End the recording and submit the recorded kernels to `stream` with one call."""
    _check(load_library().xrl_graph_launch(ctx, _stream(stream)), "xrl_graph_launch")


def xrl_launch_counts(ctx):
    a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
    _check(load_library().xrl_launch_counts(ctx, C.byref(a), C.byref(b), C.byref(c)), "xrl_launch_counts")
    return {"pack": a.value, "encode": b.value, "heads": c.value}


def xrl_profile(ctx, enable: bool):
    _check(load_library().xrl_profile(ctx, 1 if enable else 0), "xrl_profile")


def xrl_profile_read(ctx):
    n = len(PROFILE_FAMILIES)
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _check(load_library().xrl_profile_read(ctx, ms, cnt, n), "xrl_profile_read")
    return {f: {"ms": ms[i], "launches": cnt[i]} for i, f in enumerate(PROFILE_FAMILIES)}


def xrl_pack_csr_static(device, num_op_types, n_nodes, n_edges, op, edge_src, edge_dst, env_off,
                        node_off, edge_off, seg_id, graph_env, rowptr, col, device_status, stream=None):
    """Packer variant for callers that may not allocate device memory (see include/xrl.h).

    Counts and env_off are numpy int32 (host); every other array is a torch CUDA int32 tensor the
    caller allocated beforehand (inputs op/edge_src/edge_dst, outputs the packed arrays and a
    one-element status).  Nothing is allocated by the call; batches beyond the XRL_STATIC_PACK_MAX_*
    limits raise XrlError(XRL_ERR_CAPACITY).  Calls share one built-in scratch array per GPU, so
    keep them on one stream."""
    n_nodes = np.ascontiguousarray(n_nodes, dtype=np.int32)
    n_edges = np.ascontiguousarray(n_edges, dtype=np.int32)
    env_off = np.ascontiguousarray(env_off, dtype=np.int32)
    st = load_library().xrl_pack_csr_static(
        device, num_op_types, len(n_nodes), _np_ptr(n_nodes), _np_ptr(n_edges), _dev_ptr(op),
        _dev_ptr(edge_src), _dev_ptr(edge_dst), _np_ptr(env_off), len(env_off) - 1, _dev_ptr(node_off),
        _dev_ptr(edge_off), _dev_ptr(seg_id), _dev_ptr(graph_env), _dev_ptr(rowptr), _dev_ptr(col),
        _dev_ptr(device_status), _stream(stream))
    _check(st, "xrl_pack_csr_static")


# ---- the call a user makes --------------------------------------------------------------------

class Agent:
    """One model on one GPU: set weights once, then `step()` per rewrite step.

    m: dict with keys T, S, H, K, L, Hm, Dg, dtype, A_max (and optionally Hm2).  Capacities bound the
    batch size.
    """

    def __init__(self, m, max_graphs, max_envs, max_nodes, max_edges, device=0):
        import torch
        self.torch = torch
        self.m = dict(m)
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.cfg = model_config(m, max_graphs, max_envs, max_nodes, max_edges)
        self.ctx = xrl_create(self.cfg, device)
        self.batch = None
        self._out = {}
        self._steps = 0

    def close(self):
        if self.ctx is not None:
            if self.batch is not None:
                xrl_batch_free(self.ctx, self.batch)
                self.batch = None
            xrl_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_weights(self, blob):
        xrl_set_weights(self.ctx, blob)

    def _buffers(self, B, Ne):
        t = self.torch
        key = (B, Ne)
        if key not in self._out:
            self._out = {key: dict(
                emb=t.empty((B, self.m["H"]), dtype=t.float32, device=self.device),
                probs=t.empty((Ne, self.m["A_max"] + 1), dtype=t.float32, device=self.device),
                value=t.empty((Ne,), dtype=t.float32, device=self.device),
                action=t.empty((Ne,), dtype=t.int32, device=self.device))}
        return self._out[key]

    def storage_shape(self, shape_f32):
        """Host float32 shape features -> the array xrl_pack_flat expects for this model's dtype."""
        return to_bf16_bits(shape_f32) if self.m["dtype"] == "bf16" else \
            np.ascontiguousarray(shape_f32, dtype=np.float32)

    def pack(self, batch):
        """batch: flat dict (n_nodes, n_edges, op, shape, edge_src, edge_dst, env_off); bulk arrays
        either numpy (host) or torch CUDA tensors (device, shape already in storage type)."""
        on_dev = not isinstance(batch["op"], np.ndarray)
        shape = batch["shape"] if on_dev else self.storage_shape(batch["shape"])
        self.batch = xrl_pack_flat(self.ctx, XRL_MEM_DEVICE if on_dev else XRL_MEM_HOST,
                                   batch["n_nodes"], batch["n_edges"], batch["op"], shape,
                                   batch["edge_src"], batch["edge_dst"], batch["env_off"],
                                   batch=self.batch)
        if self.m.get("edge_attr"):
            ea = batch["edge_attr"]
            xrl_batch_set_edge_attr(self.ctx, self.batch, ea if on_dev else self.storage_shape(ea))
        return self.batch

    def pack_graphs(self, graphs, env_off):
        self.batch = xrl_pack(self.ctx, graphs, env_off, self.m["dtype"], batch=self.batch)
        return self.batch

    # steps with at most this many nodes are submitted as one recorded graph (their kernels are so short
    # that launching them one by one leaves the GPU waiting for the host)
    GRAPH_MAX_NODES = 65536

    def forward(self, mask, sample=False, seed=0, step=0, g0=None, base_id=None, graph=None):
        """Encode the packed batch and evaluate the heads.  mask: torch CUDA uint8 [envs, A_max].
        base_id (torch CUDA int32 [N]) switches to delta encoding of the candidates.
        graph: True submits the kernels as one recorded CUDA graph (xrl_graph_begin / xrl_graph_launch),
        False launches them one by one, None chooses by batch size (never on a context's first step, which
        also sets kernel attributes, and never with delta encoding or while profiling)."""
        info = xrl_batch_info(self.batch)
        o = self._buffers(info["num_graphs"], info["num_envs"])
        if graph is None:
            graph = self._steps > 0 and info["num_nodes"] <= self.GRAPH_MAX_NODES
        recording = False
        if graph and base_id is None:
            try:
                xrl_graph_begin(self.ctx)
                recording = True
            except XrlError as e:
                if e.status != 6:              # XRL_ERR_STATE: profiling is on, launch directly
                    raise
        try:
            if base_id is None:
                xrl_encode(self.ctx, self.batch, o["emb"], g0)
            else:
                xrl_encode_delta(self.ctx, self.batch, base_id, o["emb"], g0)
            xrl_policy_value(self.ctx, self.batch, o["emb"], mask, o["probs"], o["value"],
                             o["action"] if sample else None, seed, step)
        finally:
            if recording:
                xrl_graph_launch(self.ctx)
        self._steps += 1
        return o

    def step(self, batch, mask, sample=False, seed=0, step=0, base_id=None, graph=None):
        """The whole path for one batch: pack -> encode -> policy/value (-> sample)."""
        self.pack(batch)
        return self.forward(mask, sample, seed, step, base_id=base_id, graph=graph)

    def device_status(self):
        return xrl_last_device_status(self.ctx)

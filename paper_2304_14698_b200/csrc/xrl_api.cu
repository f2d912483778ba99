// C-ABI layer of libxrl: contexts, weights, batches and the three calls of the path
// (xrl_pack, xrl_encode, xrl_policy_value).  Host code here only validates arguments, moves
// bytes and sequences kernel launches; every step of the method runs in the kernels.
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "xrl_internal.cuh"

using namespace xrl;

// NVTX ranges (header-only; no cost unless a profiling tool has attached) around the steps of the path as they
// are enqueued: pack, Eq. 6, every attention layer's transform and aggregate, readout, Eq. 8, heads, and the
// training step.  A timeline tool shows them over the kernels they launch.
#include <cmath>
#include <nvtx3/nvToolsExt.h>

namespace {

struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

constexpr int32_t kReadoutChunkRows = 512;

struct DeviceBuf {
  void* p = nullptr;
  size_t bytes = 0;
  cudaError_t alloc(size_t n) {
    bytes = n;
    return cudaMalloc(&p, n ? n : 1);
  }
  void release() { if (p) cudaFree(p); p = nullptr; }
  template <typename T> T* as() const { return static_cast<T*>(p); }
};

size_t storage_bytes(int dtype) { return dtype == XRL_BF16 ? 2 : 4; }

}  // namespace

// Optional per-kernel-family timing: CUDA events recorded on the launching stream around every
// launcher call.  Families index the steps of the path.
enum { FAM_PACK = 0, FAM_EMBED, FAM_XFORM, FAM_AGG, FAM_READOUT, FAM_HEADS, FAM_AGG_READOUT, FAM_LAYERS, FAM_COUNT };

struct Profiler {
  bool on = false;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  struct Rec { int fam; size_t a, b; int launches; };
  std::vector<Rec> recs;
  size_t begin(cudaStream_t st) {
    if (!on) return 0;
    if (used + 2 > pool.size()) {
      cudaEvent_t e0, e1;
      if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { on = false; return 0; }
      pool.push_back(e0); pool.push_back(e1);
    }
    cudaEventRecord(pool[used], st);
    used += 2;
    return used - 2;
  }
  void end(int fam, size_t slot, int launches, cudaStream_t st) {
    if (!on) return;
    cudaEventRecord(pool[slot + 1], st);
    recs.push_back(Rec{fam, slot, slot + 1, launches});
  }
  void clear() { used = 0; recs.clear(); }
  void release() { for (cudaEvent_t e : pool) cudaEventDestroy(e); pool.clear(); clear(); }
};

struct xrl_ctx {
  Profiler prof;
  xrl_model_config cfg;
  Dims dims;
  int device = 0;
  bool weights_set = false;
  bool use_umma = false;    // bf16 transform on the tensor cores (hidden 128 or 256)
  bool use_umma_embed = false;   // bf16 node update on the tensor cores
  DeviceBuf w0ext;          // W0 extended and transposed for the tensor-core node update
  size_t weight_floats = 0;
  DeviceBuf w_f32;          // the fp32 blob
  DeviceBuf w_store;        // storage-type copies of W0 and the layer matrices (+ transposes)
  DevWeights dw;
  DeviceBuf h, Z, scores, partial, logits, status;
  DeviceBuf Z2;             // second Z buffer of the all-layers kernel for small steps (its row capacity: Z2_rows)
  int64_t Z2_rows = 0;
  int32_t max_chunks = 0;
  int64_t launches_pack = 0, launches_encode = 0, launches_heads = 0;
  // delta encoding workspace (allocated on the first xrl_encode_delta)
  DeviceBuf dl_ints, dl_col, dl_scan;
  int32_t* dl_host = nullptr;      // pinned: row counts read back per layer
  int64_t delta_rows[65] = {0};    // rows computed per layer by the last xrl_encode_delta
  // one submission per step: kernels recorded on cap_stream between xrl_graph_begin and xrl_graph_launch
  cudaStream_t cap_stream = nullptr;
  cudaGraphExec_t graph_exec = nullptr;
  bool capturing = false;
  // reverse pass: saved layer inputs and gradient scratch (allocated on the first xrl_ppo_grad)
  DeviceBuf bw;
  cudaStream_t last_pipe = nullptr;   // stream of the last batch that was packed range by range (its kernels
                                      // report bad graphs too: xrl_last_device_status waits for it as well)
};

struct xrl_batch {
  xrl_ctx* ctx = nullptr;
  bool packed = false;
  int32_t B = 0, num_envs = 0, N = 0, E = 0, num_chunks = 0;
  cudaStream_t stream = nullptr;
  // device
  DeviceBuf meta;           // n_nodes[B] n_edges[B] env_off[Ne+1] graph_chunk_off[B+1] chunk_row0[] chunk_row1[]
  DeviceBuf node_off, edge_off, seg_id, graph_env, rowptr, col, op, shape;
  DeviceBuf edge_src, edge_dst, deg, tmp_eid, long_rows, long_count, scan_ws, coarse;
  // contexts with attributes on the edges: slot -> input edge, the attributes as given and in slot order
  DeviceBuf eid, eattr_in, eattr;
  bool has_eattr = false;
  // contexts whose attention layers read neighbourhoods both ways: CSR by producer, and the merged CSR
  // (a node's producers, then its consumers) that those layers walk
  DeviceBuf rowptr_out, col_out, rowptr_nbr, col_nbr;
  const int32_t *d_n_nodes = nullptr, *d_n_edges = nullptr, *d_env_off = nullptr,
                *d_graph_chunk_off = nullptr, *d_chunk_row0 = nullptr, *d_chunk_row1 = nullptr;
  // Large batches packed from page-locked host memory are copied and packed in `nparts` ranges of whole
  // graphs on the batch's own stream `pipe`, so that the encoder can start on the first range while the
  // later ones are still crossing the bus: range p = graphs [part_g[p], part_g[p+1]) = rows
  // [part_row[p], part_row[p+1]), ready when ev_part[p] has completed.  nparts = 0: packed in one piece
  // on the caller's stream.
  static constexpr int kMaxParts = 8;
  int32_t nparts = 0;
  int32_t part_g[kMaxParts + 1] = {0}, part_row[kMaxParts + 1] = {0};
  cudaStream_t pipe = nullptr;
  cudaEvent_t ev_start = nullptr, ev_meta = nullptr, ev_part[kMaxParts] = {nullptr};
  // pinned host staging (allocated on the first pack from host memory)
  int32_t* h_meta = nullptr;
  size_t h_meta_ints = 0;
  char* h_bulk = nullptr;
  size_t h_bulk_bytes = 0;
  cudaEvent_t staged = nullptr;   // the last upload out of the staging buffers has completed
};

namespace {

xrl_status check_config(const xrl_model_config& c) {
  if (c.num_op_types < 1 || c.hidden < 1 || c.heads < 1 || c.layers < 0 || c.mlp_hidden < 1 ||
      c.global_dim < 0 || c.max_actions < 0 || c.max_graphs < 1 || c.max_envs < 1 ||
      c.max_nodes < 1 || c.max_edges < 0)
    return XRL_ERR_INVALID_ARG;
  if (c.dtype != XRL_FP32 && c.dtype != XRL_BF16) return XRL_ERR_INVALID_ARG;
  if (c.hidden % c.heads != 0) return XRL_ERR_INVALID_ARG;
  if (c.max_nodes >= (int64_t(1) << 31) - 1 || c.max_edges >= (int64_t(1) << 31) - 1)
    return XRL_ERR_INVALID_ARG;
  if (c.num_shape_feats != kS || c.num_op_types > 256) return XRL_ERR_UNSUPPORTED;
  if (c.hidden % 32 != 0 || c.hidden > 512 || (c.hidden / c.heads) % 8 != 0) return XRL_ERR_UNSUPPORTED;
  if (c.mlp_hidden2 < 0 || (c.edge_attributes != 0 && c.edge_attributes != 1) ||
      (c.neighbourhood != 0 && c.neighbourhood != 1))
    return XRL_ERR_INVALID_ARG;
  if (c.neighbourhood == 1 && c.max_edges >= (int64_t(1) << 30)) return XRL_ERR_INVALID_ARG;   // 2 E entries
  if (c.layers > 64 || c.mlp_hidden > 1024 || c.mlp_hidden2 > 1024 || c.global_dim > 16) return XRL_ERR_UNSUPPORTED;
  if (c.max_actions > (1 << 20)) return XRL_ERR_UNSUPPORTED;
  return XRL_OK;
}

size_t weight_float_count(const xrl_model_config& c) {
  const size_t S = c.num_shape_feats, T = c.num_op_types, H = c.hidden, L = c.layers,
               Hm = c.mlp_hidden, Hm2 = c.mlp_hidden2, Dg = c.global_dim;
  const size_t last = Hm2 > 0 ? Hm2 : Hm, second = Hm * Hm2 + Hm2;     // optional second hidden layer
  return (2 * S + T) * H + H + L * (H * H + 3 * H) + (H + Dg) * H + H + (H * Hm + Hm + second + last + 1) +
         (2 * H * Hm + Hm + second + last + 1);
}

#define XRL_CUDA(call)                      \
  do {                                      \
    if ((call) != cudaSuccess) {            \
      cudaGetLastError();                   \
      return XRL_ERR_CUDA;                  \
    }                                       \
  } while (0)
#define XRL_ALLOC(call)                     \
  do {                                      \
    if ((call) != cudaSuccess) {            \
      cudaGetLastError();                   \
      return XRL_ERR_ALLOC;                 \
    }                                       \
  } while (0)

xrl_status alloc_batch(xrl_ctx* ctx, xrl_batch** out) {
  xrl_batch* b = new (std::nothrow) xrl_batch();
  if (!b) return XRL_ERR_ALLOC;
  b->ctx = ctx;
  const xrl_model_config& c = ctx->cfg;
  const size_t N = size_t(c.max_nodes), E = size_t(c.max_edges), B = size_t(c.max_graphs),
               Ne = size_t(c.max_envs);
  const size_t sb = storage_bytes(c.dtype);
  b->h_meta_ints = 2 * B + (Ne + 1) + (B + 1) + 2 * size_t(ctx->max_chunks);
  cudaError_t e = cudaSuccess;
  auto A = [&](DeviceBuf& d, size_t bytes) { if (e == cudaSuccess) e = d.alloc(bytes); };
  A(b->meta, 4 * b->h_meta_ints);
  A(b->node_off, 4 * (B + 1)); A(b->edge_off, 4 * (B + 1));
  A(b->seg_id, 4 * N); A(b->graph_env, 4 * B);
  A(b->rowptr, 4 * (N + 1)); A(b->col, 4 * E);
  A(b->op, 4 * N); A(b->shape, sb * N * kS);
  A(b->edge_src, 4 * E); A(b->edge_dst, 4 * E);
  A(b->deg, 4 * N); A(b->tmp_eid, 8 * E + 8);
  A(b->long_rows, 4 * (E / 32 + 1)); A(b->long_count, 4); A(b->coarse, 4 * (E / 1024 + 2));
  A(b->scan_ws, 4 * scan_workspace_ints(int64_t(N > B ? N : B) + 1));
  if (c.edge_attributes) { A(b->eid, 4 * E); A(b->eattr_in, sb * kS * E); A(b->eattr, sb * kS * E); }
  if (c.neighbourhood) {
    A(b->rowptr_out, 4 * (N + 1)); A(b->col_out, 4 * E); A(b->rowptr_nbr, 4 * (N + 1)); A(b->col_nbr, 8 * E);
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b->staged, cudaEventDisableTiming);
  if (e != cudaSuccess) {
    cudaGetLastError();
    xrl_batch_free(ctx, b);
    return XRL_ERR_ALLOC;
  }
  *out = b;
  return XRL_OK;
}

xrl_status ensure_staging(xrl_batch* b) {
  if (b->h_meta == nullptr)
    XRL_ALLOC(cudaHostAlloc(reinterpret_cast<void**>(&b->h_meta), 4 * b->h_meta_ints, cudaHostAllocDefault));
  return XRL_OK;
}

xrl_status ensure_bulk_staging(xrl_batch* b) {
  if (b->h_bulk == nullptr) {
    const xrl_model_config& c = b->ctx->cfg;
    b->h_bulk_bytes = size_t(c.max_nodes) * (4 + storage_bytes(c.dtype) * kS) + size_t(c.max_edges) * 8;
    XRL_ALLOC(cudaHostAlloc(reinterpret_cast<void**>(&b->h_bulk), b->h_bulk_bytes ? b->h_bulk_bytes : 1,
                            cudaHostAllocDefault));
  }
  return XRL_OK;
}

// True if p is page-locked host memory (cudaHostAlloc / cudaHostRegister): asynchronous copies can
// then read it directly.  A null pointer counts as pinned (nothing to copy).
bool pinned(const void* p) {
  if (p == nullptr) return true;
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
  return a.type == cudaMemoryTypeHost;
}

// Shared tail of both pack entry points.  `graphs` non-null: gather from per-graph host arrays.
xrl_status pack_common(xrl_ctx* ctx, const xrl_graph* graphs, int32_t where, int32_t num_graphs,
                       const int32_t* n_nodes, const int32_t* n_edges, const int32_t* op,
                       const void* shape, const int32_t* edge_src, const int32_t* edge_dst,
                       const int32_t* env_off, int32_t num_envs, void* stream, xrl_batch** out) {
  if (!ctx || !out || !env_off || num_graphs < 0 || num_envs < 0) return XRL_ERR_INVALID_ARG;
  NvtxRange nvtx_pack("xrl:pack (Section 3.3.2)");
  if (ctx->capturing) return XRL_ERR_STATE;        // packing synchronises with its staging buffers
  if (!graphs && (where != XRL_MEM_HOST && where != XRL_MEM_DEVICE)) return XRL_ERR_INVALID_ARG;
  if (!graphs && num_graphs > 0 && (!n_nodes || !n_edges)) return XRL_ERR_INVALID_ARG;
  const xrl_model_config& c = ctx->cfg;
  if (num_graphs > c.max_graphs || num_envs > c.max_envs) return XRL_ERR_CAPACITY;
  if (env_off[0] != 0 || env_off[num_envs] != num_graphs) return XRL_ERR_INVALID_ARG;
  for (int32_t e = 0; e < num_envs; ++e) {
    if (env_off[e + 1] <= env_off[e]) return XRL_ERR_INVALID_ARG;
    if (env_off[e + 1] - env_off[e] - 1 > c.max_actions) return XRL_ERR_CAPACITY;
  }
  int64_t N = 0, E = 0;
  int32_t max_n = 0, max_m = 0;
  for (int32_t g = 0; g < num_graphs; ++g) {
    const int32_t n = graphs ? graphs[g].num_nodes : n_nodes[g];
    const int32_t m = graphs ? graphs[g].num_edges : n_edges[g];
    if (n < 0 || m < 0) return XRL_ERR_INVALID_ARG;
    if (n > max_n) max_n = n;
    if (m > max_m) max_m = m;
    if (graphs && ((n > 0 && (!graphs[g].op || !graphs[g].shape)) ||
                   (m > 0 && (!graphs[g].edge_src || !graphs[g].edge_dst))))
      return XRL_ERR_INVALID_ARG;
    N += n; E += m;
  }
  if (N > c.max_nodes || E > c.max_edges) return XRL_ERR_CAPACITY;
  if (!graphs && ((N > 0 && (!op || !shape)) || (E > 0 && (!edge_src || !edge_dst))))
    return XRL_ERR_INVALID_ARG;

  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  xrl_batch* b = *out;
  if (b == nullptr) {
    const xrl_status s = alloc_batch(ctx, &b);
    if (s != XRL_OK) return s;
  } else if (b->ctx != ctx) {
    return XRL_ERR_STATE;
  }
  xrl_status s = ensure_staging(b);
  const bool direct = !graphs && where == XRL_MEM_HOST && pinned(op) && pinned(shape) &&
                      pinned(edge_src) && pinned(edge_dst);
  if (s == XRL_OK && (graphs || where == XRL_MEM_HOST) && !direct) s = ensure_bulk_staging(b);
  if (s != XRL_OK) { if (*out == nullptr) xrl_batch_free(ctx, b); return s; }
  *out = b;
  b->packed = false;
  // the previous upload out of the staging buffers must have finished before they are rewritten
  XRL_CUDA(cudaEventSynchronize(b->staged));

  // ---- metadata: counts, env offsets, readout chunk list --------------------------------------
  const size_t Bz = size_t(c.max_graphs), Nez = size_t(c.max_envs);
  int32_t* m_nn = b->h_meta;
  int32_t* m_ne = m_nn + Bz;
  int32_t* m_env = m_ne + Bz;
  int32_t* m_gco = m_env + (Nez + 1);
  int32_t* m_c0 = m_gco + (Bz + 1);
  int32_t* m_c1 = m_c0 + ctx->max_chunks;
  int32_t chunks = 0, row = 0;
  for (int32_t g = 0; g < num_graphs; ++g) {
    const int32_t n = graphs ? graphs[g].num_nodes : n_nodes[g];
    m_nn[g] = n;
    m_ne[g] = graphs ? graphs[g].num_edges : n_edges[g];
    m_gco[g] = chunks;
    for (int32_t r = 0; r < n; r += kReadoutChunkRows) {
      m_c0[chunks] = row + r;
      m_c1[chunks] = row + (r + kReadoutChunkRows < n ? r + kReadoutChunkRows : n);
      ++chunks;
    }
    row += n;
  }
  m_gco[num_graphs] = chunks;
  memcpy(m_env, env_off, sizeof(int32_t) * size_t(num_envs + 1));
  XRL_CUDA(cudaMemcpyAsync(b->meta.p, b->h_meta, 4 * b->h_meta_ints, cudaMemcpyHostToDevice, st));
  const int32_t* dm = b->meta.as<int32_t>();
  b->d_n_nodes = dm; b->d_n_edges = dm + Bz; b->d_env_off = dm + 2 * Bz;
  b->d_graph_chunk_off = dm + 2 * Bz + (Nez + 1);
  b->d_chunk_row0 = b->d_graph_chunk_off + (Bz + 1);
  b->d_chunk_row1 = b->d_chunk_row0 + ctx->max_chunks;

  // ---- bulk arrays -------------------------------------------------------------------------------
  const size_t sb = storage_bytes(c.dtype);
  const int32_t *d_src, *d_dst;
  // page-locked caller memory and a large batch of graphs that the per-graph packer takes: ranges of
  // graphs are copied and packed one after the other on the batch's own stream (see xrl_batch::nparts)
  int parts = 0;
  {
    const char* ev = getenv("XRL_PIPELINE_MIN_NODES");           // testing aid: pipeline smaller batches too
    const int64_t min_nodes = ev ? atoll(ev) : (int64_t(1) << 20);
    PackIn probe{};
    probe.B = num_graphs; probe.max_n = max_n; probe.max_m = max_m;
    if (direct && num_graphs >= 2 && N >= min_nodes && min_nodes > 0 && pack_per_graph(probe) &&
        !c.neighbourhood) {                                       // (the merged CSR is built in one piece)
      const int64_t want = N / min_nodes;
      parts = int(want < 2 ? 2 : (want > xrl_batch::kMaxParts ? xrl_batch::kMaxParts : want));
      if (parts > num_graphs) parts = num_graphs;
    }
  }
  if (parts > 0 && b->pipe == nullptr) {
    XRL_CUDA(cudaStreamCreateWithFlags(&b->pipe, cudaStreamNonBlocking));
    XRL_CUDA(cudaEventCreateWithFlags(&b->ev_start, cudaEventDisableTiming));
    XRL_CUDA(cudaEventCreateWithFlags(&b->ev_meta, cudaEventDisableTiming));
    for (int p = 0; p < xrl_batch::kMaxParts; ++p)
      XRL_CUDA(cudaEventCreateWithFlags(&b->ev_part[p], cudaEventDisableTiming));
  }
  b->nparts = 0;
  if (parts > 0) {
    d_src = b->edge_src.as<int32_t>();
    d_dst = b->edge_dst.as<int32_t>();
  } else if (direct) {
    // page-locked caller memory: copy straight from it, no staging pass
    if (N) {
      XRL_CUDA(cudaMemcpyAsync(b->op.p, op, 4 * size_t(N), cudaMemcpyHostToDevice, st));
      XRL_CUDA(cudaMemcpyAsync(b->shape.p, shape, sb * kS * size_t(N), cudaMemcpyHostToDevice, st));
    }
    if (E) {
      XRL_CUDA(cudaMemcpyAsync(b->edge_src.p, edge_src, 4 * size_t(E), cudaMemcpyHostToDevice, st));
      XRL_CUDA(cudaMemcpyAsync(b->edge_dst.p, edge_dst, 4 * size_t(E), cudaMemcpyHostToDevice, st));
    }
    d_src = b->edge_src.as<int32_t>();
    d_dst = b->edge_dst.as<int32_t>();
  } else if (graphs || where == XRL_MEM_HOST) {
    char* p_op = b->h_bulk;
    char* p_shape = p_op + 4 * size_t(N);
    char* p_src = p_shape + sb * kS * size_t(N);
    char* p_dst = p_src + 4 * size_t(E);
    if (graphs) {
      size_t no = 0, eo = 0;
      for (int32_t g = 0; g < num_graphs; ++g) {
        const size_t n = size_t(graphs[g].num_nodes), m = size_t(graphs[g].num_edges);
        if (n) {
          memcpy(p_op + 4 * no, graphs[g].op, 4 * n);
          memcpy(p_shape + sb * kS * no, graphs[g].shape, sb * kS * n);
        }
        if (m) {
          memcpy(p_src + 4 * eo, graphs[g].edge_src, 4 * m);
          memcpy(p_dst + 4 * eo, graphs[g].edge_dst, 4 * m);
        }
        no += n; eo += m;
      }
    } else {
      if (N) { memcpy(p_op, op, 4 * size_t(N)); memcpy(p_shape, shape, sb * kS * size_t(N)); }
      if (E) { memcpy(p_src, edge_src, 4 * size_t(E)); memcpy(p_dst, edge_dst, 4 * size_t(E)); }
    }
    if (N) {
      XRL_CUDA(cudaMemcpyAsync(b->op.p, p_op, 4 * size_t(N), cudaMemcpyHostToDevice, st));
      XRL_CUDA(cudaMemcpyAsync(b->shape.p, p_shape, sb * kS * size_t(N), cudaMemcpyHostToDevice, st));
    }
    if (E) {
      XRL_CUDA(cudaMemcpyAsync(b->edge_src.p, p_src, 4 * size_t(E), cudaMemcpyHostToDevice, st));
      XRL_CUDA(cudaMemcpyAsync(b->edge_dst.p, p_dst, 4 * size_t(E), cudaMemcpyHostToDevice, st));
    }
    d_src = b->edge_src.as<int32_t>();
    d_dst = b->edge_dst.as<int32_t>();
  } else {
    if (N) {
      XRL_CUDA(cudaMemcpyAsync(b->op.p, op, 4 * size_t(N), cudaMemcpyDeviceToDevice, st));
      XRL_CUDA(cudaMemcpyAsync(b->shape.p, shape, sb * kS * size_t(N), cudaMemcpyDeviceToDevice, st));
    }
    d_src = edge_src;
    d_dst = edge_dst;
  }
  if (parts == 0) XRL_CUDA(cudaEventRecord(b->staged, st));

  PackIn in;
  in.B = num_graphs; in.num_envs = num_envs; in.N = int32_t(N); in.E = int32_t(E);
  in.max_n = max_n; in.max_m = max_m;
  in.n_nodes = b->d_n_nodes; in.n_edges = b->d_n_edges; in.env_off = b->d_env_off;
  in.op = b->op.as<int32_t>(); in.edge_src = d_src; in.edge_dst = d_dst;
  PackOut po;
  po.node_off = b->node_off.as<int32_t>(); po.edge_off = b->edge_off.as<int32_t>();
  po.seg_id = b->seg_id.as<int32_t>(); po.graph_env = b->graph_env.as<int32_t>();
  po.rowptr = b->rowptr.as<int32_t>(); po.col = b->col.as<int32_t>();
  po.deg = b->deg.as<int32_t>(); po.tmp_eid = b->tmp_eid.as<int32_t>();
  po.long_rows = b->long_rows.as<int32_t>(); po.long_count = b->long_count.as<int32_t>();
  po.scan_ws = b->scan_ws.as<int32_t>(); po.coarse = b->coarse.as<int32_t>();
  po.eid = c.edge_attributes ? b->eid.as<int32_t>() : nullptr;
  b->has_eattr = false;                          // attributes belong to one packing of the batch
  if (parts == 0) {
    const size_t slot = ctx->prof.begin(st);
    ctx->launches_pack = launch_pack(in, po, c.num_op_types, ctx->status.as<int32_t>(), st);
    if (c.neighbourhood) {
      // the same packing with the edges reversed gives every node's consumers; then one merged CSR
      PackIn rin = in;
      rin.edge_src = in.edge_dst; rin.edge_dst = in.edge_src;
      PackOut rpo = po;
      rpo.rowptr = b->rowptr_out.as<int32_t>(); rpo.col = b->col_out.as<int32_t>(); rpo.eid = nullptr;
      ctx->launches_pack += launch_pack(rin, rpo, c.num_op_types, ctx->status.as<int32_t>(), st);
      ctx->launches_pack += launch_merge_csr(po.rowptr, po.col, rpo.rowptr, rpo.col, in.N,
                                             b->rowptr_nbr.as<int32_t>(), b->col_nbr.as<int32_t>(), st);
    }
    ctx->prof.end(FAM_PACK, slot, int(ctx->launches_pack), st);
  } else {
    // whatever still reads the batch's arrays was queued on the caller's stream before this call
    XRL_CUDA(cudaEventRecord(b->ev_start, st));
    XRL_CUDA(cudaStreamWaitEvent(b->pipe, b->ev_start, 0));
    const size_t slot = ctx->prof.begin(st);
    int launches = launch_pack_offsets(in, po, st);            // needs the counts only
    ctx->prof.end(FAM_PACK, slot, launches, st);
    XRL_CUDA(cudaEventRecord(b->ev_meta, st));
    XRL_CUDA(cudaStreamWaitEvent(b->pipe, b->ev_meta, 0));
    // ranges of whole graphs
    const char* h_op = reinterpret_cast<const char*>(op);
    const char* h_shape = reinterpret_cast<const char*>(shape);
    int32_t g = 0;
    int64_t row = 0, edge = 0;
    b->part_g[0] = 0; b->part_row[0] = 0;
    for (int p = 0; p < parts; ++p) {
      const int64_t row0 = row, edge0 = edge;
      const int32_t g0 = g;
      // the first range is half as long as the others: nothing overlaps its copy
      const int64_t target = (N * int64_t(2 * p + 1)) / (2 * parts - 1);
      while (g < num_graphs && (p == parts - 1 || row < target || g == g0)) { row += n_nodes[g]; edge += n_edges[g]; ++g; }
      const size_t n = size_t(row - row0), m = size_t(edge - edge0);
      if (n) {
        XRL_CUDA(cudaMemcpyAsync(b->op.as<char>() + 4 * size_t(row0), h_op + 4 * size_t(row0), 4 * n,
                                 cudaMemcpyHostToDevice, b->pipe));
        XRL_CUDA(cudaMemcpyAsync(b->shape.as<char>() + sb * kS * size_t(row0), h_shape + sb * kS * size_t(row0),
                                 sb * kS * n, cudaMemcpyHostToDevice, b->pipe));
      }
      if (m) {
        XRL_CUDA(cudaMemcpyAsync(b->edge_src.as<int32_t>() + edge0, edge_src + edge0, 4 * m,
                                 cudaMemcpyHostToDevice, b->pipe));
        XRL_CUDA(cudaMemcpyAsync(b->edge_dst.as<int32_t>() + edge0, edge_dst + edge0, 4 * m,
                                 cudaMemcpyHostToDevice, b->pipe));
      }
      launches += launch_pack_graphs(in, po, c.num_op_types, g0, g, ctx->status.as<int32_t>(), b->pipe);
      XRL_CUDA(cudaEventRecord(b->ev_part[p], b->pipe));
      b->part_g[p + 1] = g; b->part_row[p + 1] = int32_t(row);
    }
    XRL_CUDA(cudaEventRecord(b->staged, b->pipe));
    b->nparts = parts;
    ctx->last_pipe = b->pipe;
    ctx->launches_pack = launches;
  }
  XRL_CUDA(cudaGetLastError());

  b->B = num_graphs; b->num_envs = num_envs; b->N = int32_t(N); b->E = int32_t(E);
  b->num_chunks = chunks; b->stream = st; b->packed = true;
  return XRL_OK;
}

// Eq. 6 and the first `layers` attention layers over the whole batch; features end up in ctx->h.
// With fuse_readout the last of the `layers` attention layers may leave per-graph partial sums in
// ctx->partial instead of node features in ctx->h; *fused tells whether it did.
// With `hs` (layers + 1 buffers of N x H storage-type values) every layer's input is kept: Eq. 6 writes hs[0],
// layer l reads hs[l] and writes hs[l + 1]; with `zs` / `ss` layer l's Z rows and half-scores go to zs[l] / ss[l]
// instead of the context's one buffer each.
int run_node_layers(xrl_ctx* ctx, const xrl_batch* b, int layers, cudaStream_t st, bool fuse_readout = false,
                    bool* fused = nullptr, int32_t row_begin = 0, int32_t row_end = -1, void* const* hs = nullptr,
                    void* const* zs = nullptr, float* const* ss = nullptr) {
  const Dims& d = ctx->dims;
  const Window win{row_begin, row_end < 0 ? b->N : row_end, 0};   // graphs are independent: any range of whole graphs
  Profiler& pf = ctx->prof;
  const void* eattr = b->has_eattr ? b->eattr.p : nullptr;      // attributes on the edges, in slot order
  // the attention layers walk the producers' CSR, or the merged one when consumers are neighbours too
  const int32_t* gat_rowptr = ctx->cfg.neighbourhood ? b->rowptr_nbr.as<int32_t>() : b->rowptr.as<int32_t>();
  const int32_t* gat_col = ctx->cfg.neighbourhood ? b->col_nbr.as<int32_t>() : b->col.as<int32_t>();
  size_t slot = pf.begin(st);
  int k = -1;
  nvtxRangePushA("xrl:node update (Eq. 6)");
  if (ctx->use_umma_embed)
    k = launch_embed_umma(d, b->rowptr.as<int32_t>(), b->col.as<int32_t>(), b->op.as<int32_t>(),
                          b->shape.p, ctx->w0ext.p, hs ? hs[0] : ctx->h.p, win, ctx->status.as<int32_t>(), st, nullptr, eattr);
  if (k < 0)
    k = launch_embed(d, b->rowptr.as<int32_t>(), b->col.as<int32_t>(), b->op.as<int32_t>(),
                     b->shape.p, ctx->dw, hs ? hs[0] : ctx->h.p, win, st, nullptr, eattr);
  pf.end(FAM_EMBED, slot, k, st);
  nvtxRangePop();
  int n = k;
  // a small step: all attention layers in one cooperative launch (same arithmetic, same outputs)
  if (!hs && !zs && !ss && win.row_begin == 0 && win.row_end == b->N && b->N <= ctx->Z2_rows && ctx->use_umma &&
      layers_coop_supported(d, layers, b->N)) {
    NvtxRange nvtx_layers("xrl:attention layers (Eq. 7), one launch");
    slot = pf.begin(st);
    k = launch_layers_coop(d, ctx->dw, layers, ctx->h.p, ctx->Z.p, ctx->Z2.p, gat_rowptr, gat_col, b->N,
                           b->seg_id.as<int32_t>(), fuse_readout ? ctx->partial.as<float>() : nullptr,
                           ctx->status.as<int32_t>(), ctx->status.as<uint32_t>() + 2, st);
    if (k >= 0) {
      pf.end(FAM_LAYERS, slot, k, st);
      if (fuse_readout && fused) *fused = true;
      return n + k;
    }
  }
  for (int l = 0; l < layers; ++l) {
    const void* h_in = hs ? hs[l] : ctx->h.p;
    void* h_out = hs ? hs[l + 1] : ctx->h.p;
    void* Zl = zs ? zs[l] : ctx->Z.p;
    float* Sl = ss ? ss[l] : ctx->scores.as<float>();
    NvtxRange nvtx_layer("xrl:attention layer (Eq. 7): transform, then score / softmax / aggregate");
    slot = pf.begin(st);
    k = -1;
    if (ctx->use_umma)
      k = launch_xform_umma(d, h_in, ctx->dw.layer[l], Zl, Sl, win,
                            ctx->status.as<int32_t>(), st);
    if (k < 0 && !d.zmerged)
      k = launch_xform_simt(d, h_in, ctx->dw.layer[l], Zl, Sl, win,
                            st);
    if (k < 0) return -1;                       // merged rows: only the tensor-core transform writes them
    pf.end(FAM_XFORM, slot, k, st);
    n += k;
    slot = pf.begin(st);
    k = -1;
    bool fused_here = false;
    if (fuse_readout && l == layers - 1) {
      k = launch_aggregate_tma(d, gat_rowptr, gat_col, Zl,
                               Sl, ctx->dw.layer[l].b, h_out, win, b->N,
                               b->seg_id.as<int32_t>(), ctx->partial.as<float>(),
                               ctx->status.as<int32_t>(), st);
      if (k >= 0) { fused_here = true; if (fused) *fused = true; }
    }
    if (k < 0)
      k = launch_aggregate(d, gat_rowptr, gat_col, Zl,
                           Sl, ctx->dw.layer[l].b,
                           h_out, win, b->N, ctx->status.as<int32_t>(), st);
    if (k < 0) return -1;
    pf.end(fused_here ? FAM_AGG_READOUT : FAM_AGG, slot, k, st);
    n += k;
  }
  return n;
}

// A batch packed range by range becomes whole for `st` once every range's event has been waited for.
xrl_status join_parts(const xrl_batch* b, cudaStream_t st) {
  for (int p = 0; p < b->nparts; ++p) XRL_CUDA(cudaStreamWaitEvent(st, b->ev_part[p], 0));
  return XRL_OK;
}

xrl_status check_batch(const xrl_ctx* ctx, const xrl_batch* b) {
  if (!ctx || !b) return XRL_ERR_INVALID_ARG;
  if (b->ctx != ctx || !b->packed || !ctx->weights_set) return XRL_ERR_STATE;
  return XRL_OK;
}

// Encoding additionally needs the edges' attributes where the model takes them from the edges.
xrl_status check_encodable(const xrl_ctx* ctx, const xrl_batch* b) {
  const xrl_status s = check_batch(ctx, b);
  if (s != XRL_OK) return s;
  if (ctx->cfg.edge_attributes && b->E > 0 && !b->has_eattr) return XRL_ERR_STATE;
  return XRL_OK;
}

}  // namespace

namespace {
template <typename F>
void grad_weigh_host(const void* grad, int64_t count, const void* loss, int64_t n, void* buf) {
  const F* g = static_cast<const F*>(grad);
  const F* l = static_cast<const F*>(loss);
  F* o = static_cast<F*>(buf);
  for (int64_t i = 0; i < count; ++i) o[i] = g[i] * F(n);
  for (int i = 0; i < 4; ++i) o[count + i] = l[i] * F(n);
  o[count + 4] = F(n);
}
template <typename F>
int64_t grad_unweigh_host(const void* buf, int64_t count, void* grad, void* loss) {
  const F* b = static_cast<const F*>(buf);
  F* g = static_cast<F*>(grad);
  F* l = static_cast<F*>(loss);
  const F total = b[count + 4];
  for (int64_t i = 0; i < count; ++i) g[i] = b[i] / total;
  for (int i = 0; i < 4; ++i) l[i] = b[count + i] / total;
  return int64_t(total + F(0.5));
}
}  // namespace

extern "C" {

const char* xrl_version(void) { return "xrl 0.1 (sm_100a, CUDA C-ABI)"; }

xrl_status xrl_create(const xrl_model_config* cfg, int32_t device, xrl_ctx** out) {
  if (!cfg || !out) return XRL_ERR_INVALID_ARG;
  *out = nullptr;
  const xrl_status s = check_config(*cfg);
  if (s != XRL_OK) return s;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return XRL_ERR_CUDA;
  }
  XRL_CUDA(cudaSetDevice(device));
  xrl_ctx* ctx = new (std::nothrow) xrl_ctx();
  if (!ctx) return XRL_ERR_ALLOC;
  ctx->cfg = *cfg;
  ctx->device = device;
  ctx->dims = Dims{cfg->num_op_types, cfg->hidden, cfg->heads, cfg->layers, cfg->mlp_hidden,
                   cfg->global_dim, cfg->max_actions, cfg->dtype, cfg->mlp_hidden2, 0};
  ctx->weight_floats = weight_float_count(*cfg);
  // XRL_FORCE_SIMT_TRANSFORM=1 keeps the CUDA-core transform for every shape (debugging aid)
  ctx->use_umma = xform_umma_supported(ctx->dims) && getenv("XRL_FORCE_SIMT_TRANSFORM") == nullptr;
  ctx->use_umma_embed = embed_umma_supported(ctx->dims) && getenv("XRL_FORCE_SIMT_TRANSFORM") == nullptr;
  // Z rows carry their half-score pairs when both kernels that touch them support it
  ctx->dims.zmerged = (ctx->use_umma && cfg->dtype == XRL_BF16 && aggregate_tma_shape(ctx->dims)) ? 1 : 0;
  ctx->max_chunks = int32_t(cfg->max_graphs + cfg->max_nodes / kReadoutChunkRows + 1);
  const size_t sb = storage_bytes(cfg->dtype), N = size_t(cfg->max_nodes), H = size_t(cfg->hidden);
  const size_t F0 = size_t(2 * kS + cfg->num_op_types);
  cudaError_t e = cudaSuccess;
  auto A = [&](DeviceBuf& d, size_t bytes) { if (e == cudaSuccess) e = d.alloc(bytes); };
  A(ctx->w_f32, 4 * ctx->weight_floats);
  A(ctx->w_store, sb * (F0 * H + 2 * size_t(cfg->layers) * H * H));
  A(ctx->w0ext, ctx->use_umma_embed ? 2 * H * size_t(embed_umma_kpad(ctx->dims)) : 0);
  A(ctx->h, sb * N * H);
  A(ctx->Z, N * z_row_bytes(ctx->dims));
  // XRL_NO_FUSED_LAYERS=1 keeps one launch per transform / attention layer for every size (debugging aid)
  if (layers_coop_supported(ctx->dims, cfg->layers > 8 ? 8 : (cfg->layers < 1 ? 1 : cfg->layers), 1) &&
      getenv("XRL_NO_FUSED_LAYERS") == nullptr) {
    ctx->Z2_rows = int64_t(N < size_t(layers_coop_max_rows()) ? N : size_t(layers_coop_max_rows()));
    A(ctx->Z2, size_t(ctx->Z2_rows) * z_row_bytes(ctx->dims));
  }
  A(ctx->scores, 8 * N * size_t(cfg->heads));
  {
    const size_t slots_fused = size_t(aggregate_readout_slots(cfg->max_nodes, cfg->max_graphs));
    const size_t slots = slots_fused > size_t(ctx->max_chunks) ? slots_fused : size_t(ctx->max_chunks);
    A(ctx->partial, 4 * slots * H);
  }
  A(ctx->logits, 4 * (size_t(cfg->max_graphs) + size_t(cfg->max_envs) * H));   // logits, then candidate sums
  A(ctx->status, 16);          // [0] the device status word; [2], [3] the all-layers kernel's barrier counters
  if (e == cudaSuccess) e = cudaMemset(ctx->status.p, 0, 16);
  if (e != cudaSuccess) {
    cudaGetLastError();
    xrl_destroy(ctx);
    return XRL_ERR_ALLOC;
  }
  *out = ctx;
  return XRL_OK;
}

void xrl_destroy(xrl_ctx* ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  DeviceBuf* bufs[] = {&ctx->w0ext, &ctx->w_f32, &ctx->w_store, &ctx->h, &ctx->Z, &ctx->scores,
                       &ctx->partial, &ctx->logits, &ctx->status, &ctx->bw, &ctx->Z2};
  for (DeviceBuf* d : bufs) d->release();
  ctx->prof.release();
  ctx->dl_ints.release(); ctx->dl_col.release(); ctx->dl_scan.release();
  if (ctx->dl_host) cudaFreeHost(ctx->dl_host);
  if (ctx->capturing) {                            // a recording left open: end it, drop the record
    cudaGraph_t g = nullptr;
    cudaStreamEndCapture(ctx->cap_stream, &g);
    if (g) cudaGraphDestroy(g);
    cudaGetLastError();
  }
  if (ctx->graph_exec) cudaGraphExecDestroy(ctx->graph_exec);
  if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
  delete ctx;
}

xrl_status xrl_weights_size(const xrl_ctx* ctx, size_t* bytes) {
  if (!ctx || !bytes) return XRL_ERR_INVALID_ARG;
  *bytes = 4 * ctx->weight_floats;
  return XRL_OK;
}

// The fp32 blob is in ctx->w_f32: derive the storage-type copies (and transposes) of W0 and the layer matrices
// and the pointers of every tensor.
static xrl_status finalize_weights(xrl_ctx* ctx) {
  const xrl_model_config& c = ctx->cfg;
  const size_t H = size_t(c.hidden), Hm = size_t(c.mlp_hidden), Hm2 = size_t(c.mlp_hidden2), Dg = size_t(c.global_dim);
  const size_t last = Hm2 > 0 ? Hm2 : Hm;
  const size_t F0 = size_t(2 * kS + c.num_op_types), sb = storage_bytes(c.dtype);
  const float* p = ctx->w_f32.as<float>();
  char* store = ctx->w_store.as<char>();
  auto take = [&](size_t n) { const float* q = p; p += n; return q; };
  DevWeights& w = ctx->dw;
  const float* W0 = take(F0 * H);
  launch_round_weights(W0, store, nullptr, int(F0), int(H), c.dtype, nullptr);
  w.W0 = store; store += sb * F0 * H;
  w.b0 = take(H);
  if (ctx->use_umma_embed) build_w0ext(ctx->dims, w.W0, w.b0, ctx->w0ext.p, nullptr);
  for (int l = 0; l < c.layers; ++l) {
    const float* W = take(H * H);
    launch_round_weights(W, store, store + sb * H * H, int(H), int(H), c.dtype, nullptr);
    w.layer[l].W = store;
    w.layer[l].Wt = store + sb * H * H;
    store += 2 * sb * H * H;
    w.layer[l].a_src = take(H);
    w.layer[l].a_dst = take(H);
    w.layer[l].b = take(H);
  }
  w.Wg = take((H + Dg) * H); w.bg = take(H);
  w.pW1 = take(H * Hm); w.pb1 = take(Hm); w.pWh = take(Hm * Hm2); w.pbh = take(Hm2);
  w.pw2 = take(last); w.pb2 = take(1);
  w.vW1 = take(2 * H * Hm); w.vb1 = take(Hm); w.vWh = take(Hm * Hm2); w.vbh = take(Hm2);
  w.vw2 = take(last); w.vb2 = take(1);
  XRL_CUDA(cudaDeviceSynchronize());
  XRL_CUDA(cudaGetLastError());
  ctx->weights_set = true;
  return XRL_OK;
}

xrl_status xrl_set_weights(xrl_ctx* ctx, const void* host_blob, size_t bytes) {
  if (!ctx || !host_blob) return XRL_ERR_INVALID_ARG;
  if (bytes != 4 * ctx->weight_floats) return XRL_ERR_INVALID_ARG;
  XRL_CUDA(cudaSetDevice(ctx->device));
  XRL_CUDA(cudaMemcpy(ctx->w_f32.p, host_blob, bytes, cudaMemcpyHostToDevice));
  return finalize_weights(ctx);
}

xrl_status xrl_init_weights(xrl_ctx* ctx, uint64_t seed) {
  if (!ctx) return XRL_ERR_INVALID_ARG;
  XRL_CUDA(cudaSetDevice(ctx->device));
  const xrl_model_config& c = ctx->cfg;
  const int64_t H = c.hidden, Hm = c.mlp_hidden, Hm2 = c.mlp_hidden2, Dg = c.global_dim;
  const int64_t F0 = 2 * kS + c.num_op_types, last = Hm2 > 0 ? Hm2 : Hm, d = H / c.heads;
  float* blob = ctx->w_f32.as<float>();
  int64_t off = 0;
  // Xavier-uniform bound sqrt(6 / (fan_in + fan_out)), taken in double and rounded to float once
  auto xavier = [](int64_t fan_in, int64_t fan_out) { return float(std::sqrt(6.0 / double(fan_in + fan_out))); };
  auto fill = [&](int64_t count, float bound) {
    launch_init_weights(blob, off, count, bound, seed, nullptr);
    off += count;
  };
  const float kBias = 0.1f;
  fill(F0 * H, xavier(F0, H)); fill(H, kBias);
  for (int l = 0; l < c.layers; ++l) {
    fill(H * H, xavier(H, H));
    fill(H, xavier(d, 1)); fill(H, xavier(d, 1));          // attention vectors: one head's width in, a score out
    fill(H, kBias);
  }
  fill((H + Dg) * H, xavier(H + Dg, H)); fill(H, kBias);
  for (int head = 0; head < 2; ++head) {                    // policy head (input H), value head (input 2 H)
    const int64_t in = head == 0 ? H : 2 * H;
    fill(in * Hm, xavier(in, Hm)); fill(Hm, kBias);
    if (Hm2 > 0) { fill(Hm * Hm2, xavier(Hm, Hm2)); fill(Hm2, kBias); }
    fill(last, xavier(last, 1)); fill(1, kBias);
  }
  if (size_t(off) != ctx->weight_floats) return XRL_ERR_STATE;
  XRL_CUDA(cudaGetLastError());
  return finalize_weights(ctx);
}

xrl_status xrl_get_weights(const xrl_ctx* ctx, void* host_blob, size_t bytes) {
  if (!ctx || !host_blob) return XRL_ERR_INVALID_ARG;
  if (bytes != 4 * ctx->weight_floats) return XRL_ERR_INVALID_ARG;
  if (!ctx->weights_set) return XRL_ERR_STATE;
  XRL_CUDA(cudaSetDevice(ctx->device));
  XRL_CUDA(cudaMemcpy(host_blob, ctx->w_f32.p, bytes, cudaMemcpyDeviceToHost));
  return XRL_OK;
}

xrl_status xrl_pack(xrl_ctx* ctx, const xrl_graph* graphs, int32_t num_graphs, const int32_t* env_off,
                    int32_t num_envs, void* stream, xrl_batch** out) {
  if (num_graphs > 0 && !graphs) return XRL_ERR_INVALID_ARG;
  static const xrl_graph none = {0, 0, nullptr, nullptr, nullptr, nullptr};
  return pack_common(ctx, graphs ? graphs : &none, XRL_MEM_HOST, num_graphs, nullptr, nullptr, nullptr,
                     nullptr, nullptr, nullptr, env_off, num_envs, stream, out);
}

xrl_status xrl_pack_flat(xrl_ctx* ctx, int32_t where, int32_t num_graphs, const int32_t* n_nodes,
                         const int32_t* n_edges, const int32_t* op, const void* shape,
                         const int32_t* edge_src, const int32_t* edge_dst, const int32_t* env_off,
                         int32_t num_envs, void* stream, xrl_batch** out) {
  return pack_common(ctx, nullptr, where, num_graphs, n_nodes, n_edges, op, shape, edge_src, edge_dst,
                     env_off, num_envs, stream, out);
}

xrl_status xrl_batch_free(xrl_ctx* ctx, xrl_batch* b) {
  if (!b) return XRL_OK;
  if (ctx && b->ctx != ctx) return XRL_ERR_STATE;
  cudaSetDevice(b->ctx->device);
  cudaDeviceSynchronize();
  DeviceBuf* bufs[] = {&b->meta, &b->node_off, &b->edge_off, &b->seg_id, &b->graph_env, &b->rowptr,
                       &b->col, &b->op, &b->shape, &b->edge_src, &b->edge_dst, &b->deg, &b->tmp_eid,
                       &b->long_rows, &b->long_count, &b->scan_ws, &b->coarse, &b->eid, &b->eattr_in,
                       &b->eattr, &b->rowptr_out, &b->col_out, &b->rowptr_nbr, &b->col_nbr};
  for (DeviceBuf* d : bufs) d->release();
  if (b->h_meta) cudaFreeHost(b->h_meta);
  if (b->h_bulk) cudaFreeHost(b->h_bulk);
  if (b->staged) cudaEventDestroy(b->staged);
  if (b->ev_start) cudaEventDestroy(b->ev_start);
  if (b->ev_meta) cudaEventDestroy(b->ev_meta);
  for (cudaEvent_t e : b->ev_part) if (e) cudaEventDestroy(e);
  if (b->pipe) {
    if (b->ctx->last_pipe == b->pipe) b->ctx->last_pipe = nullptr;
    cudaStreamDestroy(b->pipe);
  }
  delete b;
  return XRL_OK;
}

xrl_status xrl_batch_info(const xrl_batch* b, int64_t* num_nodes, int64_t* num_edges,
                          int32_t* num_graphs, int32_t* num_envs) {
  if (!b) return XRL_ERR_INVALID_ARG;
  if (!b->packed) return XRL_ERR_STATE;
  if (num_nodes) *num_nodes = b->N;
  if (num_edges) *num_edges = b->E;
  if (num_graphs) *num_graphs = b->B;
  if (num_envs) *num_envs = b->num_envs;
  return XRL_OK;
}

xrl_status xrl_batch_export(const xrl_batch* b, int32_t* rowptr, int32_t* col, int32_t* seg_id,
                            int32_t* node_off, int32_t* edge_off, int32_t* graph_env) {
  if (!b) return XRL_ERR_INVALID_ARG;
  if (!b->packed) return XRL_ERR_STATE;
  XRL_CUDA(cudaSetDevice(b->ctx->device));
  XRL_CUDA(cudaStreamSynchronize(b->stream));
  if (b->nparts > 0) XRL_CUDA(cudaStreamSynchronize(b->pipe));
  const size_t N = size_t(b->N), E = size_t(b->E), B = size_t(b->B);
  if (rowptr) XRL_CUDA(cudaMemcpy(rowptr, b->rowptr.p, 4 * (N + 1), cudaMemcpyDeviceToHost));
  if (col && E) XRL_CUDA(cudaMemcpy(col, b->col.p, 4 * E, cudaMemcpyDeviceToHost));
  if (seg_id && N) XRL_CUDA(cudaMemcpy(seg_id, b->seg_id.p, 4 * N, cudaMemcpyDeviceToHost));
  if (node_off) XRL_CUDA(cudaMemcpy(node_off, b->node_off.p, 4 * (B + 1), cudaMemcpyDeviceToHost));
  if (edge_off) XRL_CUDA(cudaMemcpy(edge_off, b->edge_off.p, 4 * (B + 1), cudaMemcpyDeviceToHost));
  if (graph_env && B) XRL_CUDA(cudaMemcpy(graph_env, b->graph_env.p, 4 * B, cudaMemcpyDeviceToHost));
  return XRL_OK;
}

xrl_status xrl_batch_set_edge_attr(xrl_ctx* ctx, xrl_batch* b, int32_t where, const void* edge_attr,
                                   void* stream) {
  if (!ctx || !b || (where != XRL_MEM_HOST && where != XRL_MEM_DEVICE)) return XRL_ERR_INVALID_ARG;
  if (b->ctx != ctx || !b->packed || !ctx->cfg.edge_attributes || ctx->capturing) return XRL_ERR_STATE;
  if (!edge_attr && b->E > 0) return XRL_ERR_INVALID_ARG;
  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  { const xrl_status js = join_parts(b, st); if (js != XRL_OK) return js; }
  const size_t row = storage_bytes(ctx->cfg.dtype) * kS, E = size_t(b->E);
  if (E > 0) {
    const void* src = edge_attr;
    if (where == XRL_MEM_HOST) {
      XRL_CUDA(cudaMemcpyAsync(b->eattr_in.p, edge_attr, row * E, cudaMemcpyHostToDevice, st));
      if (!pinned(edge_attr)) XRL_CUDA(cudaStreamSynchronize(st));     // the array is read before returning
      src = b->eattr_in.p;
    }
    launch_permute_edge_rows(src, b->eid.as<int32_t>(), b->eattr.p, int64_t(E), int(row), st);
    XRL_CUDA(cudaGetLastError());
  }
  b->has_eattr = true;
  return XRL_OK;
}

xrl_status xrl_encode(xrl_ctx* ctx, const xrl_batch* b, const float* g0, float* graph_emb, void* stream) {
  const xrl_status s = check_encodable(ctx, b);
  if (s != XRL_OK) return s;
  if (!graph_emb && b->B > 0) return XRL_ERR_INVALID_ARG;
  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = ctx->capturing ? ctx->cap_stream : static_cast<cudaStream_t>(stream);
  bool fused = false;
  NvtxRange nvtx_encode("xrl:encode (Section 3.4)");
  int n = 0;
  if (b->nparts > 0) {
    // packed range by range: encode each range of graphs as soon as it is there (the copies and the packing
    // of the later ranges run meanwhile on the batch's stream); the per-graph sums follow for all at once
    if (ctx->capturing) return XRL_ERR_STATE;
    for (int p = 0; p < b->nparts; ++p) {
      XRL_CUDA(cudaStreamWaitEvent(st, b->ev_part[p], 0));
      if (b->part_row[p + 1] == b->part_row[p]) continue;
      const int k = run_node_layers(ctx, b, ctx->cfg.layers, st, false, nullptr, b->part_row[p], b->part_row[p + 1]);
      if (k < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
      n += k;
    }
  } else {
    n = run_node_layers(ctx, b, ctx->cfg.layers, st, true, &fused);
    if (n < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
  }
  size_t slot;
  int k;
  if (!fused) {
    slot = ctx->prof.begin(st);
    k = launch_readout(ctx->dims, ctx->h.p, b->d_chunk_row0, b->d_chunk_row1, 0, b->num_chunks,
                       ctx->partial.as<float>(), 0, st);
    ctx->prof.end(FAM_READOUT, slot, k, st);
    n += k;
  }
  slot = ctx->prof.begin(st);
  if (fused)
    k = launch_global_update_blocks(ctx->dims, ctx->partial.as<float>(), b->node_off.as<int32_t>(),
                                    aggregate_readout_blocks(b->N), aggregate_block_shift(b->N), g0, ctx->dw,
                                    graph_emb, b->B, st);
  else
    k = launch_global_update(ctx->dims, ctx->partial.as<float>(), b->d_graph_chunk_off, g0, ctx->dw,
                             graph_emb, b->B, st);
  ctx->prof.end(FAM_HEADS, slot, k, st);
  n += k;
  ctx->launches_encode = n;
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_encode_delta(xrl_ctx* ctx, const xrl_batch* b, const int32_t* base_id, const float* g0,
                            float* graph_emb, void* stream) {
  const xrl_status s = check_batch(ctx, b);
  if (s != XRL_OK) return s;
  if (ctx->cfg.edge_attributes) return XRL_ERR_UNSUPPORTED;   // the node correspondence ignores edge attributes
  if (ctx->cfg.neighbourhood) return XRL_ERR_UNSUPPORTED;     // a rewrite then reaches its producers' side too
  if (ctx->capturing) return XRL_ERR_STATE;        // reads the row counts back between layers
  if (!graph_emb && b->B > 0) return XRL_ERR_INVALID_ARG;
  NvtxRange nvtx_delta("xrl:encode, delta of the candidates (Section 3.4)");
  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  { const xrl_status js = join_parts(b, st); if (js != XRL_OK) return js; }
  const size_t Ncap = size_t(ctx->cfg.max_nodes) + 1, Ecap = size_t(ctx->cfg.max_edges) + 1;
  if (ctx->dl_ints.p == nullptr) {
    XRL_ALLOC(ctx->dl_ints.alloc(4 * (10 * Ncap + 256)));
    XRL_ALLOC(ctx->dl_col.alloc(4 * Ecap));
    XRL_ALLOC(ctx->dl_scan.alloc(4 * scan_workspace_ints(int64_t(Ncap))));
    XRL_ALLOC(cudaHostAlloc(reinterpret_cast<void**>(&ctx->dl_host), 4 * 128, cudaHostAllocDefault));
  }
  int32_t* I = ctx->dl_ints.as<int32_t>();
  int32_t *valid = I, *base = I + Ncap, *level_a = I + 2 * Ncap, *level_b = I + 3 * Ncap,
          *rank = I + 4 * Ncap, *list = I + 5 * Ncap, *deg = I + 6 * Ncap, *rowptr_c = I + 7 * Ncap,
          *self_c = I + 8 * Ncap, *remap = I + 9 * Ncap, *counts = I + 10 * Ncap, *cursor = counts + 128;
  int32_t* col_c = ctx->dl_col.as<int32_t>();
  int32_t* scan_ws = ctx->dl_scan.as<int32_t>();
  const Dims& d = ctx->dims;
  const int N = b->N, L = d.L;

  DeltaIn in;
  in.N = N; in.E = b->E;
  in.seg_id = b->seg_id.as<int32_t>(); in.graph_env = b->graph_env.as<int32_t>();
  in.env_off = b->d_env_off; in.node_off = b->node_off.as<int32_t>();
  in.rowptr = b->rowptr.as<int32_t>(); in.col = b->col.as<int32_t>(); in.op = b->op.as<int32_t>();
  in.shape = b->shape.p; in.shape_bytes = int(storage_bytes(d.dtype)) * kS;
  in.base_id = base_id;

  // ---- levels, dense rows (ordered by level) and the row list ---------------------------------------
  Profiler& pf = ctx->prof;
  int n_launch = 0;
  size_t slot = pf.begin(st);
  int k = launch_delta_level0(in, valid, base, level_a, st);
  int32_t* level = level_a;
  int32_t* other = level_b;
  for (int t = 1; t <= L; ++t) {
    k += launch_delta_propagate(in, t, level, other, st);
    int32_t* tmp = level; level = other; other = tmp;
  }
  k += launch_delta_count(N, L, level, counts, cursor, st);
  k += launch_delta_assign(N, L, level, counts, cursor, rank, list, st);
  pf.end(FAM_PACK, slot, k, st);
  n_launch += k;
  // the only read-back: rows per level, which size the launches of every layer
  XRL_CUDA(cudaMemcpyAsync(ctx->dl_host, counts, 4 * size_t(L + 1), cudaMemcpyDeviceToHost, st));
  XRL_CUDA(cudaStreamSynchronize(st));
  int32_t n_at[66];
  int32_t run = 0;
  for (int t = 0; t <= L; ++t) { run += ctx->dl_host[t]; n_at[t] = run; ctx->delta_rows[t] = run; }
  const int32_t n_all = n_at[L];
  slot = pf.begin(st);
  k = launch_delta_degrees(in, n_all, list, deg, st);
  k += launch_exclusive_scan(deg, rowptr_c, n_all, scan_ws, st);
  pf.end(FAM_PACK, slot, k, st);
  n_launch += k;

  // Eq. 6 on the level-0 rows, written densely
  slot = pf.begin(st);
  const Window w0{0, n_at[0], 0};
  k = -1;
  if (ctx->use_umma_embed)
    k = launch_embed_umma(d, in.rowptr, in.col, in.op, b->shape.p, ctx->w0ext.p, ctx->h.p, w0,
                          ctx->status.as<int32_t>(), st, list);
  if (k < 0) k = launch_embed(d, in.rowptr, in.col, in.op, b->shape.p, ctx->dw, ctx->h.p, w0, st, list);
  pf.end(FAM_EMBED, slot, k, st);
  n_launch += k;

  for (int l = 0; l < L; ++l) {
    const int32_t n_prev = n_at[l], n_cur = n_at[l + 1];
    // transform of the rows reached so far (dense)
    slot = pf.begin(st);
    const Window wp{0, n_prev, 0};
    k = -1;
    if (ctx->use_umma)
      k = launch_xform_umma(d, ctx->h.p, ctx->dw.layer[l], ctx->Z.p, ctx->scores.as<float>(), wp,
                            ctx->status.as<int32_t>(), st);
    if (k < 0 && !d.zmerged)
      k = launch_xform_simt(d, ctx->h.p, ctx->dw.layer[l], ctx->Z.p, ctx->scores.as<float>(), wp, st);
    if (k < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
    pf.end(FAM_XFORM, slot, k, st);
    n_launch += k;
    // compact CSR of the rows this layer reaches: producers and the row's own vector by dense row
    slot = pf.begin(st);
    k = launch_delta_fill(in, n_cur, l + 1, list, rowptr_c, level, rank, base, col_c, self_c, st);
    pf.end(FAM_PACK, slot, k, st);
    n_launch += k;
    slot = pf.begin(st);
    const Window wc{0, n_cur, 0};
    k = launch_aggregate(d, rowptr_c, col_c, ctx->Z.p, ctx->scores.as<float>(), ctx->dw.layer[l].b, ctx->h.p,
                         wc, n_prev > 0 ? n_prev : 1, ctx->status.as<int32_t>(), st, self_c);
    if (k < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
    pf.end(FAM_AGG, slot, k, st);
    n_launch += k;
  }
  // Eq. 8: every node adds the dense row that holds its features (its own or its base node's)
  slot = pf.begin(st);
  k = launch_delta_remap(N, L, level, rank, base, remap, st);
  k += launch_readout(d, ctx->h.p, b->d_chunk_row0, b->d_chunk_row1, 0, b->num_chunks,
                      ctx->partial.as<float>(), 0, st, remap);
  pf.end(FAM_READOUT, slot, k, st);
  n_launch += k;
  slot = pf.begin(st);
  k = launch_global_update(d, ctx->partial.as<float>(), b->d_graph_chunk_off, g0, ctx->dw, graph_emb, b->B, st);
  pf.end(FAM_HEADS, slot, k, st);
  n_launch += k;
  ctx->launches_encode = n_launch;
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_delta_rows(const xrl_ctx* ctx, int64_t* rows, int32_t count) {
  if (!ctx || !rows || count < 0) return XRL_ERR_INVALID_ARG;
  for (int32_t i = 0; i < count; ++i) rows[i] = (i <= ctx->cfg.layers && i < 65) ? ctx->delta_rows[i] : 0;
  return XRL_OK;
}

xrl_status xrl_debug_node_features(xrl_ctx* ctx, const xrl_batch* b, int32_t num_layers,
                                   float* host_out, void* stream) {
  const xrl_status s = check_encodable(ctx, b);
  if (s != XRL_OK) return s;
  if (num_layers < 0 || num_layers > ctx->cfg.layers || (!host_out && b->N > 0)) return XRL_ERR_INVALID_ARG;
  if (ctx->capturing) return XRL_ERR_STATE;
  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  { const xrl_status js = join_parts(b, st); if (js != XRL_OK) return js; }
  if (run_node_layers(ctx, b, num_layers, st) < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
  const int64_t n = int64_t(b->N) * ctx->cfg.hidden;
  if (n == 0) return XRL_OK;
  float* tmp = nullptr;
  XRL_ALLOC(cudaMalloc(&tmp, sizeof(float) * size_t(n)));
  launch_to_float(ctx->h.p, ctx->cfg.dtype, tmp, n, st);
  cudaError_t e = cudaStreamSynchronize(st);
  if (e == cudaSuccess) e = cudaMemcpy(host_out, tmp, sizeof(float) * size_t(n), cudaMemcpyDeviceToHost);
  cudaFree(tmp);
  XRL_CUDA(e);
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_policy_value(xrl_ctx* ctx, const xrl_batch* b, const float* graph_emb,
                            const uint8_t* mask, float* probs, float* value, int32_t* action,
                            uint64_t seed, uint64_t step, void* stream) {
  const xrl_status s = check_batch(ctx, b);
  if (s != XRL_OK) return s;
  if (b->num_envs > 0 && (!graph_emb || !probs || !value || (!mask && ctx->cfg.max_actions > 0)))
    return XRL_ERR_INVALID_ARG;
  NvtxRange nvtx_heads("xrl:policy / value heads, masked softmax, draw (Sections 3.3.2, 3.3.3)");
  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = ctx->capturing ? ctx->cap_stream : static_cast<cudaStream_t>(stream);
  const size_t slot = ctx->prof.begin(st);
  ctx->launches_heads = launch_heads(ctx->dims, ctx->dw, graph_emb, b->d_env_off, mask, b->B, b->num_envs,
                                     ctx->logits.as<float>(), probs, value, action, seed, step,
                                     ctx->status.as<int32_t>(), st);
  ctx->prof.end(FAM_HEADS, slot, int(ctx->launches_heads), st);
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_ppo_grad(xrl_ctx* ctx, const xrl_batch* b, const float* g0, const uint8_t* mask,
                        const int32_t* action, const float* logp_old, const float* adv, const float* ret,
                        float eps, float c1, float c2, float* loss_out, float* grad, float* logp_out,
                        void* stream) {
  const xrl_status s = check_encodable(ctx, b);
  if (s != XRL_OK) return s;
  if (ctx->capturing) return XRL_ERR_STATE;
  if (!loss_out || !grad) return XRL_ERR_INVALID_ARG;
  NvtxRange nvtx_grad("xrl:training step gradient (Section 3.3.4, Eq. 3-5)");
  if (b->num_envs > 0 && (!action || !logp_old || !adv || !ret || (!mask && ctx->cfg.max_actions > 0)))
    return XRL_ERR_INVALID_ARG;
  if (embed_bwd_smem_bytes(ctx->dims) > size_t(227) * 1024) return XRL_ERR_UNSUPPORTED;
  XRL_CUDA(cudaSetDevice(ctx->device));
  const Dims& d = ctx->dims;
  const xrl_model_config& c = ctx->cfg;
  const int L = c.layers;
  auto up = [](size_t n) { return (n + 255) & ~size_t(255); };
  const size_t sb = storage_bytes(c.dtype), Nmax = size_t(c.max_nodes), H = size_t(c.hidden);
  const size_t h_bytes = up(sb * Nmax * H), f_bytes = up(4 * Nmax * H), ds_bytes = up(8 * Nmax * size_t(c.heads));
  const size_t heads_bytes = up(4 * ppo_heads_workspace_floats(d, c.max_graphs, c.max_envs));
  const size_t z_bytes = up(Nmax * z_row_bytes(d));
  if (!ctx->bw.p) {
    if (ctx->bw.alloc(size_t(L + 2) * h_bytes + size_t(L) * (z_bytes + ds_bytes) + 3 * f_bytes + ds_bytes +
                      heads_bytes) != cudaSuccess) {
      cudaGetLastError();
      ctx->bw.p = nullptr;
      return XRL_ERR_ALLOC;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (b->nparts > 0) { const xrl_status j = join_parts(b, st); if (j != XRL_OK) return j; }
  char* p = ctx->bw.as<char>();
  void* hs[65];
  for (int l = 0; l <= L; ++l) { hs[l] = p; p += h_bytes; }
  void* dz_store = p; p += h_bytes;                 // dz in the storage type, for the tensor-core products
  void* zs[64];                                     // every layer's Z rows and half-scores, kept for the reverse pass
  float* ss[64];
  for (int l = 0; l < L; ++l) { zs[l] = p; p += z_bytes; ss[l] = reinterpret_cast<float*>(p); p += ds_bytes; }
  float* dh_a = reinterpret_cast<float*>(p); p += f_bytes;
  float* dh_b = reinterpret_cast<float*>(p); p += f_bytes;
  float* dz = reinterpret_cast<float*>(p); p += f_bytes;
  float* ds = reinterpret_cast<float*>(p); p += ds_bytes;
  float* heads_ws = reinterpret_cast<float*>(p);
  XRL_CUDA(cudaMemsetAsync(grad, 0, 4 * ctx->weight_floats, st));
  XRL_CUDA(cudaMemsetAsync(loss_out, 0, 16, st));
  if (b->B == 0 || b->num_envs == 0) return XRL_OK;
  int n = run_node_layers(ctx, b, L, st, false, nullptr, 0, -1, hs, zs, ss);
  if (n < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
  const float* wb = ctx->w_f32.as<float>();
  n += launch_ppo_heads(d, ctx->dw, grad, wb, hs[L], b->node_off.as<int32_t>(), b->seg_id.as<int32_t>(), g0,
                        b->d_env_off, mask, action, logp_old, adv, ret, eps, c1, c2, b->B, b->num_envs, b->N,
                        heads_ws, loss_out, dh_a, logp_out, ctx->status.as<int32_t>(), st);
  const int32_t* gat_rowptr = c.neighbourhood ? b->rowptr_nbr.as<int32_t>() : b->rowptr.as<int32_t>();
  const int32_t* gat_col = c.neighbourhood ? b->col_nbr.as<int32_t>() : b->col.as<int32_t>();
  float* dh_cur = dh_a;
  float* dh_nxt = dh_b;
  for (int l = L - 1; l >= 0 && b->N > 0; --l) {
    const LayerWeights& lw = ctx->dw.layer[l];
    float* ga_src = grad + (lw.a_src - wb);
    const int k = launch_gat_layer_bwd(d, gat_rowptr, gat_col, zs[l], ss[l], hs[l], hs[l + 1], dh_cur,
                             dh_nxt, dz, ds, dz_store, lw, ga_src - H * H, ga_src, grad + (lw.a_dst - wb),
                             grad + (lw.b - wb), b->N, st);
    if (k < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
    n += k;
    std::swap(dh_cur, dh_nxt);
  }
  const int k = launch_embed_bwd(d, b->rowptr.as<int32_t>(), b->col.as<int32_t>(), b->op.as<int32_t>(), b->shape.p,
                                 b->has_eattr ? b->eattr.p : nullptr, hs[0], dh_cur, dz, grad,
                                 grad + (ctx->dw.b0 - wb), b->N, st);
  if (k < 0) { cudaGetLastError(); return XRL_ERR_CUDA; }
  n += k;
  (void)n;   // (launches of the reverse pass are not reported by xrl_launch_counts)
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_gae(int32_t device, int32_t num_steps, int32_t num_trajectories, const float* reward,
                   const float* values, const uint8_t* done, float gamma, float lambda, float* adv, float* ret,
                   void* stream) {
  if (num_steps < 0 || num_trajectories < 0) return XRL_ERR_INVALID_ARG;
  if (num_steps > 0 && num_trajectories > 0 && (!reward || !values || !done || !adv || !ret)) return XRL_ERR_INVALID_ARG;
  XRL_CUDA(cudaSetDevice(device));
  launch_gae(reward, values, done, gamma, lambda, num_steps, num_trajectories, adv, ret,
             static_cast<cudaStream_t>(stream));
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_grad_weigh(int32_t where, int32_t device, int32_t elem_bytes, const void* grad, int64_t count,
                          const void* loss, int64_t num_envs, void* buf, void* stream) {
  if ((where != XRL_MEM_HOST && where != XRL_MEM_DEVICE) || (elem_bytes != 4 && elem_bytes != 8) || count < 0 ||
      num_envs < 0 || !loss || !buf || (count > 0 && !grad))
    return XRL_ERR_INVALID_ARG;
  if (where == XRL_MEM_HOST) {
    if (elem_bytes == 8) grad_weigh_host<double>(grad, count, loss, num_envs, buf);
    else grad_weigh_host<float>(grad, count, loss, num_envs, buf);
    return XRL_OK;
  }
  XRL_CUDA(cudaSetDevice(device));
  launch_grad_weigh(elem_bytes, grad, count, loss, num_envs, buf, static_cast<cudaStream_t>(stream));
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_grad_unweigh(int32_t where, int32_t device, int32_t elem_bytes, const void* buf, int64_t count,
                            void* grad, void* loss, int64_t* total_envs, void* stream) {
  if ((where != XRL_MEM_HOST && where != XRL_MEM_DEVICE) || (elem_bytes != 4 && elem_bytes != 8) || count < 0 ||
      !loss || !buf || (count > 0 && !grad))
    return XRL_ERR_INVALID_ARG;
  if (where == XRL_MEM_HOST) {
    const int64_t total = elem_bytes == 8 ? grad_unweigh_host<double>(buf, count, grad, loss)
                                          : grad_unweigh_host<float>(buf, count, grad, loss);
    if (total_envs) *total_envs = total;
    return XRL_OK;
  }
  XRL_CUDA(cudaSetDevice(device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  launch_grad_unweigh(elem_bytes, buf, count, grad, loss, st);
  XRL_CUDA(cudaGetLastError());
  if (total_envs) {
    double t8 = 0.0;
    float t4 = 0.f;
    const char* last = static_cast<const char*>(buf) + size_t(count + 4) * size_t(elem_bytes);
    XRL_CUDA(cudaMemcpyAsync(elem_bytes == 8 ? static_cast<void*>(&t8) : static_cast<void*>(&t4), last,
                             size_t(elem_bytes), cudaMemcpyDeviceToHost, st));
    XRL_CUDA(cudaStreamSynchronize(st));
    *total_envs = int64_t((elem_bytes == 8 ? t8 : double(t4)) + 0.5);
  }
  return XRL_OK;
}

xrl_status xrl_sample(xrl_ctx* ctx, const float* probs, int32_t num_envs, int32_t num_actions,
                      uint64_t seed, uint64_t step, int32_t* action, void* stream) {
  if (!ctx || num_envs < 0 || num_actions < 1) return XRL_ERR_INVALID_ARG;
  if (num_envs > 0 && (!probs || !action)) return XRL_ERR_INVALID_ARG;
  XRL_CUDA(cudaSetDevice(ctx->device));
  launch_sample(probs, num_envs, num_actions, seed, step, action,
                ctx->capturing ? ctx->cap_stream : static_cast<cudaStream_t>(stream));
  XRL_CUDA(cudaGetLastError());
  return XRL_OK;
}

xrl_status xrl_last_device_status(xrl_ctx* ctx, void* stream, int32_t* status) {
  if (!ctx || !status) return XRL_ERR_INVALID_ARG;
  if (ctx->capturing) return XRL_ERR_STATE;
  XRL_CUDA(cudaSetDevice(ctx->device));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  XRL_CUDA(cudaStreamSynchronize(st));
  if (ctx->last_pipe) XRL_CUDA(cudaStreamSynchronize(ctx->last_pipe));
  XRL_CUDA(cudaMemcpy(status, ctx->status.p, 4, cudaMemcpyDeviceToHost));
  XRL_CUDA(cudaMemset(ctx->status.p, 0, 4));
  return XRL_OK;
}

xrl_status xrl_graph_begin(xrl_ctx* ctx) {
  if (!ctx) return XRL_ERR_INVALID_ARG;
  if (ctx->capturing || ctx->prof.on) return XRL_ERR_STATE;     // event timing needs direct launches
  XRL_CUDA(cudaSetDevice(ctx->device));
  if (ctx->cap_stream == nullptr)
    XRL_CUDA(cudaStreamCreateWithFlags(&ctx->cap_stream, cudaStreamNonBlocking));
  XRL_CUDA(cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeThreadLocal));
  ctx->capturing = true;
  return XRL_OK;
}

xrl_status xrl_graph_launch(xrl_ctx* ctx, void* stream) {
  if (!ctx) return XRL_ERR_INVALID_ARG;
  if (!ctx->capturing) return XRL_ERR_STATE;
  ctx->capturing = false;
  cudaSetDevice(ctx->device);
  cudaGraph_t graph = nullptr;
  if (cudaStreamEndCapture(ctx->cap_stream, &graph) != cudaSuccess || graph == nullptr) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    return XRL_ERR_CUDA;
  }
  bool ready = false;
  if (ctx->graph_exec != nullptr) {                // same kernel sequence as last time: update in place
    cudaGraphExecUpdateResultInfo info;
    if (cudaGraphExecUpdate(ctx->graph_exec, graph, &info) == cudaSuccess) {
      ready = true;
    } else {
      cudaGetLastError();
      cudaGraphExecDestroy(ctx->graph_exec);
      ctx->graph_exec = nullptr;
    }
  }
  cudaError_t e = cudaSuccess;
  if (!ready) e = cudaGraphInstantiate(&ctx->graph_exec, graph, 0);
  if (e == cudaSuccess) e = cudaGraphLaunch(ctx->graph_exec, static_cast<cudaStream_t>(stream));
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) { cudaGetLastError(); return XRL_ERR_CUDA; }
  return XRL_OK;
}

xrl_status xrl_profile(xrl_ctx* ctx, int32_t enable) {
  if (!ctx) return XRL_ERR_INVALID_ARG;
  if (ctx->capturing) return XRL_ERR_STATE;
  XRL_CUDA(cudaSetDevice(ctx->device));
  XRL_CUDA(cudaDeviceSynchronize());
  ctx->prof.clear();
  ctx->prof.on = enable != 0;
  return XRL_OK;
}

xrl_status xrl_profile_read(xrl_ctx* ctx, double* total_ms, int64_t* launches, int32_t num_families) {
  if (!ctx || !total_ms || !launches || num_families < 0) return XRL_ERR_INVALID_ARG;
  if (ctx->capturing) return XRL_ERR_STATE;
  XRL_CUDA(cudaSetDevice(ctx->device));
  XRL_CUDA(cudaDeviceSynchronize());
  for (int f = 0; f < num_families; ++f) { total_ms[f] = 0.0; launches[f] = 0; }
  for (const Profiler::Rec& r : ctx->prof.recs) {
    float ms = 0.f;
    XRL_CUDA(cudaEventElapsedTime(&ms, ctx->prof.pool[r.a], ctx->prof.pool[r.b]));
    if (r.fam < num_families) { total_ms[r.fam] += ms; launches[r.fam] += r.launches; }
  }
  ctx->prof.clear();
  return XRL_OK;
}

xrl_status xrl_launch_counts(const xrl_ctx* ctx, int64_t* pack, int64_t* encode, int64_t* heads) {
  if (!ctx) return XRL_ERR_INVALID_ARG;
  if (pack) *pack = ctx->launches_pack;
  if (encode) *encode = ctx->launches_encode;
  if (heads) *heads = ctx->launches_heads;
  return XRL_OK;
}

}  // extern "C"

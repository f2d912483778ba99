// Delta encoding of candidates (the paper's candidates are the current graph with one rewrite applied at
// one location, Section 3.2 / 3.3.1): a candidate node whose operator, shape features and producers
// equal those of a node of its environment's current graph, and whose producers are themselves
// unchanged, has the same features as that node at layer 0; a change reaches a node one attention
// layer after it reached one of its producers.  These kernels find, per layer, the rows that have to be
// computed ("dirty"), list them, and build the compact CSR that lets the ordinary encoder kernels run on
// the listed rows only, reading every unchanged producer from the current graph's row instead.
// Integer-only; the caller's base_id is a hint that is verified here, so a wrong hint costs time, not
// correctness.
#include "xrl_internal.cuh"

namespace xrl {

namespace {

constexpr int TB = 256;

// valid[i] = 1 iff i is a candidate node whose hint points at a node of its environment's current graph
// with the same operator and bit-identical shape features; base[i] = that node, else -1.
// Nodes of current graphs are never valid (they are always computed).
__global__ void k_delta_valid(DeltaIn in, int32_t* __restrict__ valid, int32_t* __restrict__ base) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= in.N) return;
  const int32_t g = in.seg_id[i];
  const int32_t gcur = in.env_off[in.graph_env[g]];
  int32_t ok = 0, b = -1;
  if (g != gcur && in.base_id != nullptr) {
    b = in.base_id[i];
    if (b >= in.node_off[gcur] && b < in.node_off[gcur + 1] && in.op[i] == in.op[b]) {
      const uint32_t* si = reinterpret_cast<const uint32_t*>(static_cast<const char*>(in.shape) + size_t(i) * in.shape_bytes);
      const uint32_t* sb = reinterpret_cast<const uint32_t*>(static_cast<const char*>(in.shape) + size_t(b) * in.shape_bytes);
      ok = 1;
      for (int w = 0; w < in.shape_bytes / 4; ++w) ok &= (si[w] == sb[w]) ? 1 : 0;
    }
  }
  valid[i] = ok;
  base[i] = ok ? b : -1;
}

// Layer-0 dirtiness: not valid, or the producer list differs from the base node's (same length, and
// producer k is a valid node whose base is the base node's producer k).
__global__ void k_delta_dirty0(DeltaIn in, const int32_t* __restrict__ valid, const int32_t* __restrict__ base,
                               int32_t* __restrict__ flag) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= in.N) return;
  int32_t dirty = 1;
  if (valid[i]) {
    const int32_t b = base[i];
    const int32_t e0 = in.rowptr[i], n = in.rowptr[i + 1] - e0;
    const int32_t f0 = in.rowptr[b];
    if (n == in.rowptr[b + 1] - f0) {
      dirty = 0;
      for (int32_t k = 0; k < n; ++k) {
        const int32_t j = in.col[e0 + k];
        if (!valid[j] || base[j] != in.col[f0 + k]) { dirty = 1; break; }
      }
    }
  }
  flag[i] = dirty;
}

// One attention layer later: dirty if it was, or if any producer was.
__global__ void k_delta_propagate(DeltaIn in, const int32_t* __restrict__ fin, int32_t* __restrict__ fout) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= in.N) return;
  int32_t d = fin[i];
  for (int32_t e = in.rowptr[i]; e < in.rowptr[i + 1] && !d; ++e) d = fin[in.col[e]];
  fout[i] = d;
}

__global__ void k_delta_list(int32_t N, const int32_t* __restrict__ flag, const int32_t* __restrict__ rank,
                             int32_t* __restrict__ list) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N && flag[i]) list[rank[i]] = i;
}

__global__ void k_delta_degrees(DeltaIn in, int32_t n, const int32_t* __restrict__ list,
                                int32_t* __restrict__ deg) {
  const int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n) return;
  const int32_t i = list[r];
  deg[r] = in.rowptr[i + 1] - in.rowptr[i];
}

// Row of the dense Z buffer of this layer that holds node j's vector: its own if it was recomputed,
// else the row of the current-graph node it equals.
__device__ __forceinline__ int32_t dense_row(int32_t j, const int32_t* __restrict__ flag_prev,
                                             const int32_t* __restrict__ rank_prev,
                                             const int32_t* __restrict__ base) {
  return flag_prev[j] ? rank_prev[j] : rank_prev[base[j]];
}

__global__ void k_delta_fill(DeltaIn in, int32_t n, const int32_t* __restrict__ list,
                             const int32_t* __restrict__ rowptr_c, const int32_t* __restrict__ flag_prev,
                             const int32_t* __restrict__ rank_prev, const int32_t* __restrict__ base,
                             int32_t* __restrict__ col_c, int32_t* __restrict__ self_c) {
  const int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n) return;
  const int32_t i = list[r];
  self_c[r] = dense_row(i, flag_prev, rank_prev, base);
  const int32_t e0 = in.rowptr[i], m = in.rowptr[i + 1] - e0, o = rowptr_c[r];
  for (int32_t k = 0; k < m; ++k) col_c[o + k] = dense_row(in.col[e0 + k], flag_prev, rank_prev, base);
}

__global__ void k_delta_remap(int32_t N, const int32_t* __restrict__ flag, const int32_t* __restrict__ rank,
                              const int32_t* __restrict__ base, int32_t* __restrict__ remap) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) remap[i] = dense_row(i, flag, rank, base);
}

inline int grid(int64_t n) { return int((n + TB - 1) / TB); }

}  // namespace

int launch_delta_init(const DeltaIn& in, int32_t* valid, int32_t* base, int32_t* flag0, cudaStream_t st) {
  if (in.N <= 0) return 0;
  k_delta_valid<<<grid(in.N), TB, 0, st>>>(in, valid, base);
  k_delta_dirty0<<<grid(in.N), TB, 0, st>>>(in, valid, base, flag0);
  return 2;
}
int launch_delta_propagate(const DeltaIn& in, const int32_t* flag_in, int32_t* flag_out, cudaStream_t st) {
  if (in.N <= 0) return 0;
  k_delta_propagate<<<grid(in.N), TB, 0, st>>>(in, flag_in, flag_out);
  return 1;
}
int launch_delta_list(int32_t N, const int32_t* flag, const int32_t* rank, int32_t* list, cudaStream_t st) {
  if (N <= 0) return 0;
  k_delta_list<<<grid(N), TB, 0, st>>>(N, flag, rank, list);
  return 1;
}
int launch_delta_degrees(const DeltaIn& in, int32_t n, const int32_t* list, int32_t* deg, cudaStream_t st) {
  if (n <= 0) return 0;
  k_delta_degrees<<<grid(n), TB, 0, st>>>(in, n, list, deg);
  return 1;
}
int launch_delta_fill(const DeltaIn& in, int32_t n, const int32_t* list, const int32_t* rowptr_c,
                      const int32_t* flag_prev, const int32_t* rank_prev, const int32_t* base,
                      int32_t* col_c, int32_t* self_c, cudaStream_t st) {
  if (n <= 0) return 0;
  k_delta_fill<<<grid(n), TB, 0, st>>>(in, n, list, rowptr_c, flag_prev, rank_prev, base, col_c, self_c);
  return 1;
}
int launch_delta_remap(int32_t N, const int32_t* flag, const int32_t* rank, const int32_t* base,
                       int32_t* remap, cudaStream_t st) {
  if (N <= 0) return 0;
  k_delta_remap<<<grid(N), TB, 0, st>>>(N, flag, rank, base, remap);
  return 1;
}

}  // namespace xrl

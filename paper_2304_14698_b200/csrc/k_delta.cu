// Delta encoding of candidates (the paper's candidates are the current graph with one rewrite applied at
// one location, Section 3.2 / 3.3.1): a candidate node whose operator, shape features and producers
// equal those of a node of its environment's current graph, and whose producers are themselves
// unchanged, has the same features as that node at layer 0; a change reaches a node one attention
// layer after it reached one of its producers.  These kernels find, per layer, the rows that have to be
// computed ("dirty"), list them, and build the compact CSR that lets the ordinary encoder kernels run on
// the listed rows only, reading every unchanged producer from the current graph's row instead.
// Every reached node gets a level (the layer at which the change reaches it) and one dense row for all
// layers, rows ordered by level: layer t then works on a prefix of the row list.  Integer-only; the
// caller's base_id is a hint that is verified here, so a wrong hint costs time, not correctness.
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

constexpr int32_t kNever = 1 << 20;   // level of a node no change reaches within the layers

// level[i] = 0 if the node has to be computed from Eq. 6 on: not valid, or the producer list differs
// from the base node's (same length, and producer k is a valid node whose base is the base node's
// producer k); kNever otherwise (for now).
__global__ void k_delta_level0(DeltaIn in, const int32_t* __restrict__ valid, const int32_t* __restrict__ base,
                               int32_t* __restrict__ level) {
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
  level[i] = dirty ? 0 : kNever;
}

// One attention layer later: a node not reached so far is reached at layer t if one of its producers was
// reached before (Eq. 7 reads producers only).  Reads lin, writes lout (no in-place update: the level of
// a node must not depend on the order in which threads run).
__global__ void k_delta_propagate(DeltaIn in, int32_t t, const int32_t* __restrict__ lin,
                                  int32_t* __restrict__ lout) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= in.N) return;
  int32_t lv = lin[i];
  if (lv == kNever)
    for (int32_t e = in.rowptr[i]; e < in.rowptr[i + 1]; ++e)
      if (lin[in.col[e]] < t) { lv = t; break; }
  lout[i] = lv;
}

// counts[v] = number of nodes with level v (v <= L); warp-aggregated atomics
__global__ void k_delta_count(int32_t N, const int32_t* __restrict__ level, int32_t* __restrict__ counts) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  const int32_t lv = (i < N) ? level[i] : kNever;
  const uint32_t peers = __match_any_sync(0xFFFFFFFFu, lv);
  if (lv != kNever && (threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&counts[lv], __popc(peers));
}

// Dense row of every reached node: rows are ordered by level (inside a level in whatever order the
// atomics give: the row order changes no result, rows are computed independently and summed per graph
// in node order).  cursor[v] must be zero on entry; offset of level v = counts[0] + ... + counts[v-1].
__global__ void k_delta_assign(int32_t N, int32_t L, const int32_t* __restrict__ level,
                               const int32_t* __restrict__ counts, int32_t* __restrict__ cursor,
                               int32_t* __restrict__ rank, int32_t* __restrict__ list) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  const int32_t lv = (i < N) ? level[i] : kNever;
  const uint32_t peers = __match_any_sync(0xFFFFFFFFu, lv);
  if (lv == kNever) return;
  const int lane = threadIdx.x & 31, leader = __ffs(peers) - 1;
  int32_t start = 0;
  if (lane == leader) {
    for (int32_t v = 0; v < lv; ++v) start += counts[v];
    start += atomicAdd(&cursor[lv], __popc(peers));
  }
  start = __shfl_sync(peers, start, leader);
  const int32_t r = start + __popc(peers & ((1u << lane) - 1u));
  rank[i] = r;
  list[r] = i;
  (void)L;
}

__global__ void k_delta_degrees(DeltaIn in, int32_t n, const int32_t* __restrict__ list,
                                int32_t* __restrict__ deg) {
  const int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n) return;
  const int32_t i = list[r];
  deg[r] = in.rowptr[i + 1] - in.rowptr[i];
}

// Row of the dense buffers that holds node j's vector when layer `t` reads it: its own if a change had
// reached it before (level < t), else the row of the current-graph node it equals (always level 0).
__device__ __forceinline__ int32_t dense_row(int32_t j, int32_t t, const int32_t* __restrict__ level,
                                             const int32_t* __restrict__ rank, const int32_t* __restrict__ base) {
  return level[j] < t ? rank[j] : rank[base[j]];
}

// Compact CSR of the first n listed rows for attention layer t (1-based)
__global__ void k_delta_fill(DeltaIn in, int32_t n, int32_t t, const int32_t* __restrict__ list,
                             const int32_t* __restrict__ rowptr_c, const int32_t* __restrict__ level,
                             const int32_t* __restrict__ rank, const int32_t* __restrict__ base,
                             int32_t* __restrict__ col_c, int32_t* __restrict__ self_c) {
  const int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n) return;
  const int32_t i = list[r];
  self_c[r] = dense_row(i, t, level, rank, base);
  const int32_t e0 = in.rowptr[i], m = in.rowptr[i + 1] - e0, o = rowptr_c[r];
  for (int32_t k = 0; k < m; ++k) col_c[o + k] = dense_row(in.col[e0 + k], t, level, rank, base);
}

// where each node's final features live (for the per-graph sum)
__global__ void k_delta_remap(int32_t N, int32_t L, const int32_t* __restrict__ level,
                              const int32_t* __restrict__ rank, const int32_t* __restrict__ base,
                              int32_t* __restrict__ remap) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) remap[i] = dense_row(i, L + 1, level, rank, base);
}

inline int grid(int64_t n) { return int((n + TB - 1) / TB); }

}  // namespace

int launch_delta_level0(const DeltaIn& in, int32_t* valid, int32_t* base, int32_t* level, cudaStream_t st) {
  if (in.N <= 0) return 0;
  k_delta_valid<<<grid(in.N), TB, 0, st>>>(in, valid, base);
  k_delta_level0<<<grid(in.N), TB, 0, st>>>(in, valid, base, level);
  return 2;
}
int launch_delta_propagate(const DeltaIn& in, int32_t t, const int32_t* level_in, int32_t* level_out,
                           cudaStream_t st) {
  if (in.N <= 0) return 0;
  k_delta_propagate<<<grid(in.N), TB, 0, st>>>(in, t, level_in, level_out);
  return 1;
}
// counts / cursor: [L + 2] ints each, zeroed here
int launch_delta_count(int32_t N, int32_t L, const int32_t* level, int32_t* counts, int32_t* cursor,
                       cudaStream_t st) {
  cudaMemsetAsync(counts, 0, sizeof(int32_t) * size_t(L + 2), st);
  cudaMemsetAsync(cursor, 0, sizeof(int32_t) * size_t(L + 2), st);
  if (N <= 0) return 0;
  k_delta_count<<<grid(N), TB, 0, st>>>(N, level, counts);
  return 1;
}
int launch_delta_assign(int32_t N, int32_t L, const int32_t* level, const int32_t* counts, int32_t* cursor,
                        int32_t* rank, int32_t* list, cudaStream_t st) {
  if (N <= 0) return 0;
  k_delta_assign<<<grid(N), TB, 0, st>>>(N, L, level, counts, cursor, rank, list);
  return 1;
}
int launch_delta_degrees(const DeltaIn& in, int32_t n, const int32_t* list, int32_t* deg, cudaStream_t st) {
  if (n <= 0) return 0;
  k_delta_degrees<<<grid(n), TB, 0, st>>>(in, n, list, deg);
  return 1;
}
int launch_delta_fill(const DeltaIn& in, int32_t n, int32_t t, const int32_t* list, const int32_t* rowptr_c,
                      const int32_t* level, const int32_t* rank, const int32_t* base, int32_t* col_c,
                      int32_t* self_c, cudaStream_t st) {
  if (n <= 0) return 0;
  k_delta_fill<<<grid(n), TB, 0, st>>>(in, n, t, list, rowptr_c, level, rank, base, col_c, self_c);
  return 1;
}
int launch_delta_remap(int32_t N, int32_t L, const int32_t* level, const int32_t* rank, const int32_t* base,
                       int32_t* remap, cudaStream_t st) {
  if (N <= 0) return 0;
  k_delta_remap<<<grid(N), TB, 0, st>>>(N, L, level, rank, base, remap);
  return 1;
}

}  // namespace xrl

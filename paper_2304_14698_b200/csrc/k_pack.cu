// Meta-graph packer (paper Section 3.3.2: the current graph and its candidates are batched
// into one graph).  Integer-only, deterministic: exclusive scans for the per-graph offsets,
// segment ids, in-degree count, and a CSR-by-consumer fill that keeps, inside every row, the
// order of the input edge list.
#include "xrl_internal.cuh"

namespace xrl {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;                       // per thread
constexpr int kScanTile = kScanThreads * kScanItems;

// Exclusive scan of one tile; in[i] is taken as 0 for i >= n_in; writes out[i] for i < n_out.
// If block_sums != nullptr the tile total goes there.
__global__ void __launch_bounds__(kScanThreads)
k_scan_tile(const int32_t* __restrict__ in, int32_t* __restrict__ out, int32_t n_in, int32_t n_out,
            int32_t* __restrict__ block_sums) {
  __shared__ int32_t warp_tot[kScanThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int64_t base = int64_t(blockIdx.x) * kScanTile + int64_t(tid) * kScanItems;
  int32_t v[kScanItems];
  int32_t sum = 0;
#pragma unroll
  for (int t = 0; t < kScanItems; ++t) {
    const int64_t i = base + t;
    v[t] = (i < n_in) ? in[i] : 0;
    sum += v[t];
  }
  int32_t incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) warp_tot[wid] = incl;
  __syncthreads();
  int32_t warp_base = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kScanThreads / 32; ++w) {
    if (w < wid) warp_base += warp_tot[w];
    total += warp_tot[w];
  }
  int32_t run = warp_base + incl - sum;
#pragma unroll
  for (int t = 0; t < kScanItems; ++t) {
    const int64_t i = base + t;
    if (i < n_out) out[i] = run;
    run += v[t];
  }
  if (block_sums != nullptr && tid == 0) block_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kScanThreads)
k_scan_add(int32_t* __restrict__ out, int32_t n_out, const int32_t* __restrict__ block_offsets) {
  const int32_t add = block_offsets[blockIdx.x];
  const int64_t base = int64_t(blockIdx.x) * kScanTile + int64_t(threadIdx.x) * kScanItems;
#pragma unroll
  for (int t = 0; t < kScanItems; ++t)
    if (base + t < n_out) out[base + t] += add;
}

int num_tiles(int64_t n) { return int((n + kScanTile - 1) / kScanTile); }

// out[0..n_in] = exclusive scan of in[0..n_in) (n_in + 1 outputs, the last is the total).
// ws holds the per-tile sums of every level.
int exclusive_scan(const int32_t* in, int32_t* out, int32_t n_in, int32_t* ws, cudaStream_t st) {
  const int32_t n_out = n_in + 1;
  const int tiles = num_tiles(n_out);
  int launches = 0;
  if (tiles == 1) {
    k_scan_tile<<<1, kScanThreads, 0, st>>>(in, out, n_in, n_out, nullptr);
    return 1;
  }
  int32_t* sums = ws;
  int32_t* sums_scanned = ws + tiles;
  k_scan_tile<<<tiles, kScanThreads, 0, st>>>(in, out, n_in, n_out, sums);
  ++launches;
  // scan of the tile sums (tiles outputs are enough; the recursion writes tiles + 1)
  launches += exclusive_scan(sums, sums_scanned, tiles, ws + 2 * tiles + 2, st);
  k_scan_add<<<tiles, kScanThreads, 0, st>>>(out, n_out, sums_scanned);
  return launches + 1;
}

__device__ __forceinline__ int32_t upper_segment(const int32_t* __restrict__ off, int32_t n_seg,
                                                 int32_t x) {
  // largest g in [0, n_seg) with off[g] <= x  (off is non-decreasing, off[0] = 0)
  int32_t lo = 0, hi = n_seg;
  while (hi - lo > 1) {
    const int32_t mid = (lo + hi) >> 1;
    if (__ldg(off + mid) <= x) lo = mid; else hi = mid;
  }
  return lo;
}

// Graph of every 1024-th edge: lets the per-edge kernels find their graph with a short forward walk
// instead of a binary search.
constexpr int kCoarseShift = 10;
__global__ void k_edge_coarse(const int32_t* __restrict__ edge_off, int32_t B, int32_t E,
                              int32_t* __restrict__ coarse) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if ((int64_t(i) << kCoarseShift) < E) coarse[i] = upper_segment(edge_off, B, i << kCoarseShift);
}
__device__ __forceinline__ int32_t graph_of_edge(const int32_t* __restrict__ edge_off,
                                                 const int32_t* __restrict__ coarse, int32_t B, int32_t e) {
  int32_t g = __ldg(coarse + (e >> kCoarseShift));
  while (g + 1 < B && __ldg(edge_off + g + 1) <= e) ++g;      // skips empty graphs as well
  return g;
}

__global__ void k_node_segments(const int32_t* __restrict__ node_off, int32_t B, int32_t N,
                                const int32_t* __restrict__ op, int32_t T,
                                int32_t* __restrict__ seg_id, int32_t* __restrict__ deg,
                                int32_t* status) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  seg_id[i] = upper_segment(node_off, B, i);
  deg[i] = 0;
  const int32_t o = op[i];
  if (o < 0 || o >= T) raise(status, XRL_ERR_BAD_GRAPH);
}

__global__ void k_graph_envs(const int32_t* __restrict__ env_off, int32_t num_envs, int32_t B,
                             int32_t* __restrict__ graph_env) {
  const int32_t g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g < B) graph_env[g] = upper_segment(env_off, num_envs, g);
}

// One thread per edge: validate, count the consumer's in-degree.
__global__ void k_edge_count(const int32_t* __restrict__ edge_src, const int32_t* __restrict__ edge_dst,
                             const int32_t* __restrict__ edge_off, const int32_t* __restrict__ node_off,
                             const int32_t* __restrict__ coarse, int32_t B, int32_t E,
                             int32_t* __restrict__ deg, int32_t* status) {
  const int32_t e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  const int32_t g = graph_of_edge(edge_off, coarse, B, e);
  const int32_t n = node_off[g + 1] - node_off[g];
  const int32_t s = edge_src[e], t = edge_dst[e];
  if (s < 0 || s >= n || t < 0 || t >= n || s == t) { raise(status, XRL_ERR_BAD_GRAPH); return; }
  atomicAdd(&deg[node_off[g] + t], 1);
}

// One thread per edge: drop (edge id, global producer id) into some slot of its consumer's row
// (the order inside the row is fixed later from the edge ids).
__global__ void k_edge_scatter(const int32_t* __restrict__ edge_src, const int32_t* __restrict__ edge_dst,
                               const int32_t* __restrict__ edge_off, const int32_t* __restrict__ node_off,
                               const int32_t* __restrict__ coarse, const int32_t* __restrict__ rowptr,
                               int32_t B, int32_t E, int32_t* __restrict__ cursor,
                               int2* __restrict__ tmp) {
  const int32_t e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  const int32_t g = graph_of_edge(edge_off, coarse, B, e);
  const int32_t n = node_off[g + 1] - node_off[g];
  const int32_t s = edge_src[e], t = edge_dst[e];
  if (s < 0 || s >= n || t < 0 || t >= n || s == t) return;
  const int32_t row = node_off[g] + t;
  const int32_t slot = atomicAdd(&cursor[row], 1);
  tmp[rowptr[row] + slot] = make_int2(e, node_off[g] + s);
}

constexpr int kShortRow = 32;

// One thread per row: place each producer at the rank of its edge id among the row's edge ids, which
// restores the input order whatever order the atomics handed the slots out in.
// eid (optional): the input edge that lands in each slot, for attributes that live on the edges.
__global__ void k_row_order(const int32_t* __restrict__ rowptr, const int2* __restrict__ tmp, int32_t N,
                            int32_t* __restrict__ col, int32_t* __restrict__ long_rows,
                            int32_t* __restrict__ long_count, int32_t* __restrict__ eid) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int32_t b = rowptr[i], n = rowptr[i + 1] - b;
  if (n == 0) return;
  if (n == 1) { col[b] = tmp[b].y; if (eid) eid[b] = tmp[b].x; return; }
  if (n > kShortRow) { long_rows[atomicAdd(long_count, 1)] = i; return; }
  for (int32_t a = 0; a < n; ++a) {
    const int2 ea = tmp[b + a];
    int32_t rank = 0;
    for (int32_t c = 0; c < n; ++c) rank += (tmp[b + c].x < ea.x) ? 1 : 0;
    col[b + rank] = ea.y;
    if (eid) eid[b + rank] = ea.x;
  }
}

// Rows longer than kShortRow: one warp per row, the same rank computation spread over lanes.
__global__ void __launch_bounds__(256)
k_row_order_long(const int32_t* __restrict__ rowptr, const int2* __restrict__ tmp,
                 int32_t* __restrict__ col, const int32_t* __restrict__ long_rows,
                 const int32_t* __restrict__ long_count, int32_t* __restrict__ eid) {
  const int lane = threadIdx.x & 31;
  const int32_t warps = (gridDim.x * blockDim.x) >> 5;
  const int32_t count = *long_count;
  for (int32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < count; w += warps) {
    const int32_t i = long_rows[w];
    const int32_t b = rowptr[i], n = rowptr[i + 1] - b;
    for (int32_t a = lane; a < n; a += 32) {
      const int2 ea = tmp[b + a];
      int32_t rank = 0;
      for (int32_t c = 0; c < n; ++c) rank += (tmp[b + c].x < ea.x) ? 1 : 0;
      col[b + rank] = ea.y;
      if (eid) eid[b + rank] = ea.x;
    }
  }
}

// ---- one CTA per graph: the whole CSR of a graph built in shared memory ---------------------------
// For graphs whose counters and edge slots fit in shared memory: in-degrees by shared-memory atomics, a
// block scan, a scatter of (edge id, producer) pairs into the rows and the per-row rank restore all stay
// on chip; global memory sees each edge once on the way in and each output once on the way out.  Rows of
// graph g occupy col[edge_off[g] .. edge_off[g+1]), so no scan over all nodes is needed.
// Threads per graph: 1,024 for graphs of thousands of nodes (one CTA per SM fits anyway: more threads hide
// more latency), 512 for smaller graphs (several CTAs share an SM).
constexpr int kGraphThreadsMax = 1024;
inline int graph_threads(int32_t max_n) { return max_n >= 2048 ? 1024 : 512; }

// OFFSETS = true (small batches, one launch for the whole batch): the CTA also derives its graph's offsets
// from the per-graph counts itself (a block-wide sum over the graphs before it) and writes node_off[g],
// edge_off[g] and graph_env[g] (the last graph's CTA the closing entries too), which saves the three tiny
// launches that otherwise build them first.
template <int NT, bool OFFSETS>
__global__ void __launch_bounds__(NT)
k_pack_graph(int32_t* __restrict__ node_off, int32_t* __restrict__ edge_off,
             const int32_t* __restrict__ op, const int32_t* __restrict__ edge_src,
             const int32_t* __restrict__ edge_dst, int32_t T, int32_t B, int32_t cap_n,
             int32_t* __restrict__ seg_id, int32_t* __restrict__ rowptr, int32_t* __restrict__ col,
             int32_t* status, int32_t g_first, int32_t* __restrict__ eid,
             const int32_t* __restrict__ n_nodes, const int32_t* __restrict__ n_edges,
             const int32_t* __restrict__ env_off, int32_t num_envs, int32_t* __restrict__ graph_env) {
  extern __shared__ __align__(16) int32_t psm[];
  int32_t* deg = psm;                         // [cap_n + 1] in-degree, then exclusive row starts
  int32_t* cur = psm + cap_n + 1;             // [cap_n]     row cursors
  int32_t* wsum = cur + cap_n;                // [kGraphThreadsMax / 32 + 1]
  int2* tmp = reinterpret_cast<int2*>(wsum + kGraphThreadsMax / 32 + 3);   // word 2 cap_n + 20: 8-byte aligned
  const int32_t g = g_first + blockIdx.x;      // a launch may cover a range of the batch's graphs
  const int tid = threadIdx.x;
  int32_t nb, n, eb, m;
  if (OFFSETS) {
    // nodes and edges of the graphs before this one: per-thread partial sums, then a sum over the block
    int32_t sn = 0, se = 0;
    for (int32_t i = tid; i < g; i += NT) { sn += __ldg(n_nodes + i); se += __ldg(n_edges + i); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      sn += __shfl_xor_sync(0xFFFFFFFFu, sn, o);
      se += __shfl_xor_sync(0xFFFFFFFFu, se, o);
    }
    if ((tid & 31) == 0) wsum[tid >> 5] = sn;
    __syncthreads();
    sn = 0;
    for (int w = 0; w < NT / 32; ++w) sn += wsum[w];
    __syncthreads();
    if ((tid & 31) == 0) wsum[tid >> 5] = se;
    __syncthreads();
    se = 0;
    for (int w = 0; w < NT / 32; ++w) se += wsum[w];
    __syncthreads();
    nb = sn; eb = se;
    n = __ldg(n_nodes + g); m = __ldg(n_edges + g);
    if (tid == 0) {
      node_off[g] = nb; edge_off[g] = eb;
      if (g == B - 1) { node_off[B] = nb + n; edge_off[B] = eb + m; }
      graph_env[g] = upper_segment(env_off, num_envs, g);
    }
  } else {
    nb = node_off[g]; n = node_off[g + 1] - nb;
    eb = edge_off[g]; m = edge_off[g + 1] - eb;
  }

  for (int32_t i = tid; i < n; i += NT) {
    deg[i] = 0;
    cur[i] = 0;
    seg_id[nb + i] = g;
    const int32_t o = op[nb + i];
    if (o < 0 || o >= T) raise(status, XRL_ERR_BAD_GRAPH);
  }
  __syncthreads();
  // edges four at a time per thread: the loads of a batch are issued before any of them is used
  for (int32_t e0 = tid; e0 < m; e0 += 4 * NT) {
    int32_t s[4], t[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int32_t e = e0 + u * NT;
      s[u] = e < m ? __ldg(edge_src + eb + e) : 0;
      t[u] = e < m ? __ldg(edge_dst + eb + e) : -2;          // -2: no edge here
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (t[u] == -2) continue;
      if (s[u] < 0 || s[u] >= n || t[u] < 0 || t[u] >= n || s[u] == t[u]) raise(status, XRL_ERR_BAD_GRAPH);
      else atomicAdd(&deg[t[u]], 1);
    }
  }
  __syncthreads();
  // exclusive scan of deg[0..n): each thread scans a contiguous slice, warp / block offsets on top
  const int32_t per = (n + NT - 1) / NT;
  const int32_t a0 = min(n, tid * per), a1 = min(n, a0 + per);
  int32_t sum = 0;
  for (int32_t i = a0; i < a1; ++i) sum += deg[i];
  int32_t incl = sum;
  const int lane = tid & 31, wid = tid >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) wsum[wid] = incl;
  __syncthreads();
  int32_t wbase = 0;
  for (int w = 0; w < wid; ++w) wbase += wsum[w];
  int32_t run = wbase + incl - sum;
  for (int32_t i = a0; i < a1; ++i) { const int32_t dgr = deg[i]; deg[i] = run; run += dgr; }
  if (tid == NT - 1) deg[n] = run;          // valid edges of the graph
  __syncthreads();
  for (int32_t i = tid; i < n; i += NT) rowptr[nb + i] = eb + deg[i];
  if (g == B - 1 && tid == 0) rowptr[nb + n] = eb + deg[n];
  // the last graph of a partial launch closes its last row itself (the next graph's CTA, which writes the
  // same value as its first row start, may run much later)
  else if (blockIdx.x == gridDim.x - 1 && tid == 0) rowptr[nb + n] = eb + m;
  // A malformed graph (already reported through `status`) keeps fewer edges than it was given slots for:
  // the slots left over sit at the end of the last row before the next graph's rows and nobody writes them.
  // They get a valid node id (the graph's first node) so that a batch that is encoded although it was
  // reported bad still reads inside the arrays.
  if (deg[n] < m) {
    const int32_t fill = n > 0 ? nb : 0;
    for (int32_t i = deg[n] + tid; i < m; i += NT) {
      col[eb + i] = fill;
      if (eid) eid[eb + i] = eb;
    }
  }
  // scatter (edge id, global producer) into the rows, slot order as the atomics hand it out
  for (int32_t e0 = tid; e0 < m; e0 += 4 * NT) {
    int32_t s[4], t[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int32_t e = e0 + u * NT;
      s[u] = e < m ? __ldg(edge_src + eb + e) : 0;
      t[u] = e < m ? __ldg(edge_dst + eb + e) : -2;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (t[u] == -2 || s[u] < 0 || s[u] >= n || t[u] < 0 || t[u] >= n || s[u] == t[u]) continue;
      tmp[deg[t[u]] + atomicAdd(&cur[t[u]], 1)] = make_int2(e0 + u * NT, nb + s[u]);
    }
  }
  __syncthreads();
  // rank of each edge id inside its row restores the input order; short rows by one thread ...
  for (int32_t i = tid; i < n; i += NT) {
    const int32_t b = deg[i], k = deg[i + 1] - b;
    if (k == 1) { col[eb + b] = tmp[b].y; if (eid) eid[eb + b] = eb + tmp[b].x; }
    else if (k > 1 && k <= kShortRow)
      for (int32_t a = 0; a < k; ++a) {
        const int2 ea = tmp[b + a];
        int32_t rank = 0;
        for (int32_t c = 0; c < k; ++c) rank += (tmp[b + c].x < ea.x) ? 1 : 0;
        col[eb + b + rank] = ea.y;
        if (eid) eid[eb + b + rank] = eb + ea.x;      // edge ids are local to the graph in here
      }
  }
  // ... long rows by one warp each
  for (int32_t i = wid; i < n; i += NT / 32) {
    const int32_t b = deg[i], k = deg[i + 1] - b;
    if (k <= kShortRow) continue;
    for (int32_t a = lane; a < k; a += 32) {
      const int2 ea = tmp[b + a];
      int32_t rank = 0;
      for (int32_t c = 0; c < k; ++c) rank += (tmp[b + c].x < ea.x) ? 1 : 0;
      col[eb + b + rank] = ea.y;
      if (eid) eid[eb + b + rank] = eb + ea.x;
    }
  }
}

size_t pack_graph_smem(int32_t cap_n, int32_t cap_m) {
  return 4 * size_t(2 * cap_n + 1 + kGraphThreadsMax / 32 + 3) + 8 * size_t(cap_m) + 16;
}

}  // namespace

// Attributes on the edges, brought from input edge order into CSR slot order: dst[k] = src[eid[k]], rows of
// `row_bytes` bytes (a multiple of 16), one 16-byte piece per thread.
namespace {
__global__ void k_permute_rows(const uint4* __restrict__ src, const int32_t* __restrict__ eid,
                               uint4* __restrict__ dst, int64_t E, int pieces) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= E * pieces) return;
  const int64_t k = i / pieces;
  const int p = int(i - k * pieces);
  dst[i] = __ldg(src + int64_t(__ldg(eid + k)) * pieces + p);
}
}  // namespace

int launch_permute_edge_rows(const void* src, const int32_t* eid, void* dst, int64_t E, int row_bytes,
                             cudaStream_t st) {
  if (E <= 0) return 0;
  const int pieces = row_bytes / 16;
  const int64_t n = E * pieces;
  k_permute_rows<<<unsigned((n + 255) / 256), 256, 0, st>>>(static_cast<const uint4*>(src), eid,
                                                             static_cast<uint4*>(dst), E, pieces);
  return 1;
}

// Neighbourhoods read both ways: row i of the merged CSR = row i of the CSR by consumer (i's producers),
// then row i of the CSR by producer (i's consumers).  One thread per row copies both pieces.
namespace {
__global__ void k_merge_csr(const int32_t* __restrict__ rp_a, const int32_t* __restrict__ col_a,
                            const int32_t* __restrict__ rp_b, const int32_t* __restrict__ col_b, int32_t N,
                            int32_t* __restrict__ rp_m, int32_t* __restrict__ col_m) {
  const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i > N) return;
  const int32_t a0 = rp_a[i], b0 = rp_b[i];
  rp_m[i] = a0 + b0;
  if (i == N) return;
  const int32_t na = rp_a[i + 1] - a0, nb = rp_b[i + 1] - b0;
  int32_t* dst = col_m + a0 + b0;
  for (int32_t t = 0; t < na; ++t) dst[t] = col_a[a0 + t];
  for (int32_t t = 0; t < nb; ++t) dst[na + t] = col_b[b0 + t];
}
}  // namespace

int launch_merge_csr(const int32_t* rp_a, const int32_t* col_a, const int32_t* rp_b, const int32_t* col_b,
                     int32_t N, int32_t* rp_m, int32_t* col_m, cudaStream_t st) {
  k_merge_csr<<<(N + 1 + 255) / 256, 256, 0, st>>>(rp_a, col_a, rp_b, col_b, N, rp_m, col_m);
  return 1;
}

int launch_exclusive_scan(const int32_t* in, int32_t* out, int32_t n_in, int32_t* ws, cudaStream_t st) {
  return exclusive_scan(in, out, n_in, ws, st);
}

size_t scan_workspace_ints(int64_t n) {
  size_t total = 0;
  int64_t m = n + 1;
  while (true) {
    const int64_t tiles = (m + kScanTile - 1) / kScanTile;
    if (tiles <= 1) break;
    total += size_t(2 * tiles + 2);
    m = tiles + 1;
  }
  return total + 16;
}

// Graphs small enough for shared memory: one CTA builds the whole CSR of a graph.
bool pack_per_graph(const PackIn& in) {
  return in.B > 0 && in.max_n > 0 && in.max_n <= 16384 && pack_graph_smem(in.max_n, in.max_m) <= 160 * 1024;
}

// Offsets and graph -> environment table: needs the per-graph counts only, not the graphs themselves.
int launch_pack_offsets(const PackIn& in, const PackOut& out, cudaStream_t st) {
  int launches = 0;
  const int TB = 256;
  launches += exclusive_scan(in.n_nodes, out.node_off, in.B, out.scan_ws, st);
  launches += exclusive_scan(in.n_edges, out.edge_off, in.B, out.scan_ws, st);
  if (in.B > 0) {
    k_graph_envs<<<(in.B + TB - 1) / TB, TB, 0, st>>>(in.env_off, in.num_envs, in.B, out.graph_env);
    ++launches;
  }
  return launches;
}

// CSR, segment ids and validation of graphs [g0, g1) (pack_per_graph(in) must hold; offsets already built, or
// with `offsets` built by the same launch, which must then cover the whole batch).
int launch_pack_graphs(const PackIn& in, const PackOut& out, int T, int32_t g0, int32_t g1, int32_t* status,
                       cudaStream_t st, bool offsets) {
  if (g1 <= g0) return 0;
  static bool attr512[64] = {}, attr1024[64] = {}, attr512o[64] = {}, attr1024o[64] = {};
  const size_t smem = pack_graph_smem(in.max_n, in.max_m);
#define PACK_GRAPH(NT_, OFF_, ATTR_)                                                                              \
  do {                                                                                                            \
    ensure_dynamic_smem(k_pack_graph<NT_, OFF_>, 160 * 1024, ATTR_);                                              \
    k_pack_graph<NT_, OFF_><<<g1 - g0, NT_, smem, st>>>(out.node_off, out.edge_off, in.op, in.edge_src,           \
                                                        in.edge_dst, T, in.B, in.max_n, out.seg_id, out.rowptr,   \
                                                        out.col, status, g0, out.eid, in.n_nodes, in.n_edges,     \
                                                        in.env_off, in.num_envs, out.graph_env);                  \
  } while (0)
  if (graph_threads(in.max_n) == 1024) {
    if (offsets) PACK_GRAPH(1024, true, attr1024o); else PACK_GRAPH(1024, false, attr1024);
  } else {
    if (offsets) PACK_GRAPH(512, true, attr512o); else PACK_GRAPH(512, false, attr512);
  }
#undef PACK_GRAPH
  return 1;
}

// Batches of few graphs: the per-graph kernel builds the offsets too (one launch instead of four).
constexpr int32_t kSelfOffsetGraphs = 2048;

int launch_pack(const PackIn& in, const PackOut& out, int T, int32_t* status, cudaStream_t st) {
  if (pack_per_graph(in) && in.B <= kSelfOffsetGraphs) return launch_pack_graphs(in, out, T, 0, in.B, status, st, true);
  int launches = launch_pack_offsets(in, out, st);
  const int TB = 256;
  if (pack_per_graph(in)) return launches + launch_pack_graphs(in, out, T, 0, in.B, status, st);
  if (in.N > 0) {
    k_node_segments<<<(in.N + TB - 1) / TB, TB, 0, st>>>(out.node_off, in.B, in.N, in.op, T,
                                                          out.seg_id, out.deg, status);
    ++launches;
  }
  if (in.E > 0) {
    const int nc = (in.E >> kCoarseShift) + 1;
    k_edge_coarse<<<(nc + TB - 1) / TB, TB, 0, st>>>(out.edge_off, in.B, in.E, out.coarse);
    k_edge_count<<<(in.E + TB - 1) / TB, TB, 0, st>>>(in.edge_src, in.edge_dst, out.edge_off,
                                                       out.node_off, out.coarse, in.B, in.E, out.deg, status);
    launches += 2;
  }
  launches += exclusive_scan(out.deg, out.rowptr, in.N, out.scan_ws, st);
  if (in.E > 0 && in.N > 0) {
    cudaMemsetAsync(out.deg, 0, sizeof(int32_t) * size_t(in.N), st);      // reused as the row cursors
    cudaMemsetAsync(out.long_count, 0, sizeof(int32_t), st);
    int2* tmp = reinterpret_cast<int2*>(out.tmp_eid);
    k_edge_scatter<<<(in.E + TB - 1) / TB, TB, 0, st>>>(in.edge_src, in.edge_dst, out.edge_off,
                                                         out.node_off, out.coarse, out.rowptr, in.B, in.E,
                                                         out.deg, tmp);
    k_row_order<<<(in.N + TB - 1) / TB, TB, 0, st>>>(out.rowptr, tmp, in.N, out.col, out.long_rows,
                                                      out.long_count, out.eid);
    k_row_order_long<<<kNumSMs, 256, 0, st>>>(out.rowptr, tmp, out.col, out.long_rows, out.long_count, out.eid);
    launches += 3;
  }
  return launches;
}

}  // namespace xrl

// ---- packing without any allocation -----------------------------------------------------------
// Scratch for xrl_pack_csr_static lives in the library image instead of in memory obtained at run
// time.  Layout (int32 words): n_nodes[G] n_edges[G] env_off[V+1] deg[N] tmp[2E] long_rows[E/32+1]
// long_count[1] scan workspace[kStaticScanInts] coarse[E/1024+1], with G/V/N/E the maxima below.
namespace {

constexpr int64_t kStG = XRL_STATIC_PACK_MAX_GRAPHS, kStV = XRL_STATIC_PACK_MAX_ENVS,
                  kStN = XRL_STATIC_PACK_MAX_NODES, kStE = XRL_STATIC_PACK_MAX_EDGES;
constexpr int64_t kStaticScanInts = 1024;
constexpr int64_t kOffNn = 0, kOffNe = kOffNn + kStG, kOffEnv = kOffNe + kStG, kOffDeg = kOffEnv + kStV + 1,
                  kOffTmp = (kOffDeg + kStN + 1) & ~int64_t(1) /* 8-byte aligned pairs */,
                  kOffLong = kOffTmp + 2 * kStE,
                  kOffCount = kOffLong + kStE / 32 + 1, kOffScan = kOffCount + 1,
                  kOffCoarse = kOffScan + kStaticScanInts, kStaticInts = kOffCoarse + (kStE >> 10) + 1;

static __device__ __align__(256) int32_t g_pack_scratch[kStaticInts];

constexpr int kMaxDevices = 64;
int32_t* g_pack_scratch_addr[kMaxDevices] = {};   // device address of the array, per device

}  // namespace

extern "C" xrl_status xrl_pack_csr_static(int32_t device, int32_t num_op_types, int32_t num_graphs,
                                          const int32_t* n_nodes, const int32_t* n_edges,
                                          const int32_t* op, const int32_t* edge_src,
                                          const int32_t* edge_dst, const int32_t* env_off,
                                          int32_t num_envs, int32_t* node_off, int32_t* edge_off,
                                          int32_t* seg_id, int32_t* graph_env, int32_t* rowptr,
                                          int32_t* col, int32_t* device_status, void* stream) {
  using namespace xrl;
  if (device < 0 || device >= kMaxDevices || num_op_types < 1 || num_graphs < 0 || num_envs < 0 ||
      !env_off || !node_off || !edge_off || !rowptr || !device_status ||
      (num_graphs > 0 && (!n_nodes || !n_edges || !graph_env)))
    return XRL_ERR_INVALID_ARG;
  if (num_graphs > kStG || num_envs > kStV) return XRL_ERR_CAPACITY;
  if (env_off[0] != 0 || env_off[num_envs] != num_graphs) return XRL_ERR_INVALID_ARG;
  for (int32_t e = 0; e < num_envs; ++e)
    if (env_off[e + 1] <= env_off[e]) return XRL_ERR_INVALID_ARG;
  int64_t N = 0, E = 0;
  int32_t max_n = 0, max_m = 0;
  for (int32_t g = 0; g < num_graphs; ++g) {
    if (n_nodes[g] < 0 || n_edges[g] < 0) return XRL_ERR_INVALID_ARG;
    N += n_nodes[g]; E += n_edges[g];
    if (n_nodes[g] > max_n) max_n = n_nodes[g];
    if (n_edges[g] > max_m) max_m = n_edges[g];
  }
  if (N > kStN || E > kStE) return XRL_ERR_CAPACITY;          // beyond the built-in scratch
  if ((N > 0 && (!op || !seg_id)) || (E > 0 && (!edge_src || !edge_dst || !col))) return XRL_ERR_INVALID_ARG;
  if (scan_workspace_ints((N > num_graphs ? N : num_graphs) + 1) > size_t(kStaticScanInts))
    return XRL_ERR_CAPACITY;

  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return XRL_ERR_CUDA; }
  if (g_pack_scratch_addr[device] == nullptr) {
    // one-time set-up on this device: the array's name is only a host-side handle, kernels need
    // the address the device sees
    int32_t* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_pack_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return XRL_ERR_CUDA;
    }
    g_pack_scratch_addr[device] = p;
  }
  int32_t* sc = g_pack_scratch_addr[device];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(device_status, 0, sizeof(int32_t), st);
  if (e == cudaSuccess && num_graphs > 0) {
    e = cudaMemcpyAsync(sc + kOffNn, n_nodes, 4 * size_t(num_graphs), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(sc + kOffNe, n_edges, 4 * size_t(num_graphs), cudaMemcpyHostToDevice, st);
  }
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(sc + kOffEnv, env_off, 4 * size_t(num_envs + 1), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) { cudaGetLastError(); return XRL_ERR_CUDA; }

  PackIn in;
  in.B = num_graphs; in.num_envs = num_envs; in.N = int32_t(N); in.E = int32_t(E);
  in.max_n = max_n; in.max_m = max_m;
  in.n_nodes = sc + kOffNn; in.n_edges = sc + kOffNe; in.env_off = sc + kOffEnv;
  in.op = op; in.edge_src = edge_src; in.edge_dst = edge_dst;
  PackOut out;
  out.node_off = node_off; out.edge_off = edge_off; out.seg_id = seg_id; out.graph_env = graph_env;
  out.rowptr = rowptr; out.col = col;
  out.deg = sc + kOffDeg; out.tmp_eid = sc + kOffTmp; out.long_rows = sc + kOffLong;
  out.long_count = sc + kOffCount; out.scan_ws = sc + kOffScan; out.coarse = sc + kOffCoarse;
  // the pack kernels zero what they count into (deg, the row cursors, long_count) themselves
  launch_pack(in, out, num_op_types, device_status, st);
  if (cudaGetLastError() != cudaSuccess) return XRL_ERR_CUDA;
  return XRL_OK;
}

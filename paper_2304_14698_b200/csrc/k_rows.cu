// Row-wise kernels of the encoder (paper Section 3.4): the node-update layer (Eq. 6), the
// attention half-scores, and the edge-score / segment-softmax / weighted-aggregate step of a
// graph-attention layer (Eq. 7).  One group of LPR lanes owns one destination row and moves it
// as 16-byte vectors (VPL vectors per lane); 32 / LPR rows share a warp.
#include "xrl_internal.cuh"

namespace xrl {

namespace {

constexpr int kRowThreads = 256;

// 8 shape features of one node as floats (all lanes of a group read the same address).
__device__ __forceinline__ void load_shape(const float* shape, int32_t node, float (&f)[kS]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(shape + size_t(node) * kS));
  const float4 b = __ldg(reinterpret_cast<const float4*>(shape + size_t(node) * kS) + 1);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
__device__ __forceinline__ void load_shape(const bf16* shape, int32_t node, float (&f)[kS]) {
  unpack(__ldg(reinterpret_cast<const uint4*>(shape + size_t(node) * kS)), f);
}

// ---- Eq. 6: h0_i = ReLU(W0^T [ sum_{j->i} shape_j | onehot(op_i) | shape_i ] + b0) -----------
// (with attributes on the edges, Section 3.3.2 as written, the sum runs over the in-edges' own attributes)
// The one-hot block of the product is a row lookup of W0; the two shape blocks are a 16 x H
// dense map kept in shared memory as fp32.  A warp takes 8 rows at a time in two phases: first a lane per row
// gathers the row's sixteen dense inputs (row pointers, producers, their shape features: a chain of dependent
// loads, 8 chains side by side), then the warp's lanes share each row's columns, reading the inputs back from
// shared memory; the lookups of W0 for up to four rows are issued before the first is used.
constexpr int kEmbedWarps = kRowThreads / 32;
constexpr int kEmbedRows = 8;        // rows a warp takes at a time
struct EmbedStage { float x[kEmbedRows][2 * kS]; int32_t op[kEmbedRows]; };

template <typename T, int LPR, int VPL>
__global__ void __launch_bounds__(kRowThreads)
k_embed(const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
        const int32_t* __restrict__ op, const T* __restrict__ shape, const T* __restrict__ W0,
        const float* __restrict__ b0, T* __restrict__ h, int H, int Tn, Window win,
        const int32_t* __restrict__ row_list, const T* __restrict__ eattr) {
  constexpr int VEC = VecOf<T>::N;
  constexpr int RPW = 32 / LPR;
  extern __shared__ __align__(16) float smem[];
  EmbedStage& stg = reinterpret_cast<EmbedStage*>(smem)[threadIdx.x >> 5];
  float* Wd = smem + kEmbedWarps * (sizeof(EmbedStage) / sizeof(float));   // [2*kS][H]
  float* bs = Wd + 2 * kS * H;                                             // [H]
  for (int t = threadIdx.x; t < 2 * kS * H; t += blockDim.x) {
    const int s = t / H, c = t - s * H;
    const int src_row = (s < kS) ? s : (kS + Tn + (s - kS));
    Wd[t] = to_float(W0[size_t(src_row) * H + c]);
  }
  for (int t = threadIdx.x; t < H; t += blockDim.x) bs[t] = b0[t];
  __syncthreads();

  const int NV = H / VEC;
  const int lane = threadIdx.x & 31, sub = lane / LPR, sl = lane % LPR;
  const int warps_total = (gridDim.x * blockDim.x) >> 5;
  const int warp_id = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  // fp32 rows with one vector of columns per lane: the lane's 16 x VEC slice of the dense map and its bias stay in registers
  // (read from shared memory per row, the map makes the kernel wait on shared-memory bandwidth)
  constexpr bool REGW = VPL == 1 && VEC == 4;
  float wreg[REGW ? 2 * kS : 1][VEC], breg[VEC];
  if (REGW && sl < NV) {
#pragma unroll
    for (int s = 0; s < 2 * kS; ++s)
#pragma unroll
      for (int t = 0; t < VEC; ++t) wreg[REGW ? s : 0][t] = Wd[s * H + sl * VEC + t];
#pragma unroll
    for (int t = 0; t < VEC; ++t) breg[t] = bs[sl * VEC + t];
  }
  for (int64_t r0 = int64_t(win.row_begin) + int64_t(warp_id) * kEmbedRows; r0 < win.row_end;
       r0 += int64_t(warps_total) * kEmbedRows) {
    const int nr = int(min(int64_t(kEmbedRows), win.row_end - r0));
    __syncwarp();
    if (lane < nr) {
      const int32_t out_row = int32_t(r0) + lane;
      const int32_t row = row_list ? __ldg(row_list + out_row) : out_row;   // listed rows are written densely
      float x[kS];
#pragma unroll
      for (int s = 0; s < kS; ++s) x[s] = 0.f;
      const int32_t e0 = __ldg(rowptr + row), e1 = __ldg(rowptr + row + 1);
      for (int32_t e = e0; e < e1; ++e) {
        float f[kS];
        if (eattr) load_shape(eattr, e, f);            // attributes on the edges, already in slot order
        else load_shape(shape, __ldg(col + e), f);     // the producer's shape features
#pragma unroll
        for (int s = 0; s < kS; ++s) x[s] += f[s];
      }
      float own[kS];
      load_shape(shape, row, own);
#pragma unroll
      for (int s = 0; s < kS; ++s) { stg.x[lane][s] = x[s]; stg.x[lane][kS + s] = own[s]; }
      // an operator id outside the table was reported by the packer; clamped here so that nothing is read
      // outside W0 if the caller encodes such a batch anyway
      stg.op[lane] = min(max(__ldg(op + row), 0), Tn - 1);
    }
    __syncwarp();
    constexpr int U = (VPL >= 4) ? 1 : (VPL == 2 ? 2 : 4);     // rows whose lookups are in flight together
    for (int rb = sub; rb < nr; rb += RPW * U) {
      float acc[U][VPL][VEC];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int rr = rb + u * RPW;
        if (rr < nr) {
          const T* lookup = W0 + size_t(kS + stg.op[rr]) * H;
#pragma unroll
          for (int v = 0; v < VPL; ++v) {
            const int vi = v * LPR + sl;
            if (vi < NV) load_vec(lookup + vi * VEC, acc[u][v]);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int rr = rb + u * RPW;
        if (rr >= nr) continue;
        float x[2 * kS];
#pragma unroll
        for (int s = 0; s < 2 * kS; s += 4) {
          const float4 v4 = *reinterpret_cast<const float4*>(&stg.x[rr][s]);
          x[s] = v4.x; x[s + 1] = v4.y; x[s + 2] = v4.z; x[s + 3] = v4.w;
        }
        T* out = h + size_t(int32_t(r0) + rr - win.win_base) * H;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
          const int vi = v * LPR + sl;
          if (vi < NV) {
            const int c0 = vi * VEC;
            if (REGW) {
#pragma unroll
              for (int t = 0; t < VEC; ++t) acc[u][v][t] += breg[t];
#pragma unroll
              for (int s = 0; s < 2 * kS; ++s)
#pragma unroll
                for (int t = 0; t < VEC; ++t) acc[u][v][t] = fmaf(x[s], wreg[REGW ? s : 0][t], acc[u][v][t]);
            } else {
#pragma unroll
              for (int t = 0; t < VEC; ++t) acc[u][v][t] += bs[c0 + t];
#pragma unroll
              for (int s = 0; s < 2 * kS; ++s)
#pragma unroll
                for (int t = 0; t < VEC; ++t) acc[u][v][t] = fmaf(x[s], Wd[s * H + c0 + t], acc[u][v][t]);
            }
#pragma unroll
            for (int t = 0; t < VEC; ++t) acc[u][v][t] = fmaxf(acc[u][v][t], 0.f);
            store_vec(out + c0, acc[u][v]);
          }
        }
      }
    }
  }
}

// ---- attention half-scores from Z (used when the transform kernel does not emit them) ------
// s_src[i,k] = log2(e) a_src[k] . Z[i, head k],  s_dst[i,k] = log2(e) a_dst[k] . Z[i, head k]
// (stored pre-multiplied by log2(e): the aggregate kernel then needs exp2 only)
template <typename T, int LPR, int VPL>
__global__ void __launch_bounds__(kRowThreads)
k_scores(const T* __restrict__ Z, const float* __restrict__ a_src, const float* __restrict__ a_dst,
         float2* __restrict__ scores, int H, int K, Window win) {
  constexpr int VEC = VecOf<T>::N;
  constexpr int RPW = 32 / LPR;
  constexpr int WARPS = kRowThreads / 32;
  __shared__ float part[WARPS][RPW][LPR * VPL][2];
  const int NV = H / VEC, d = H / K, vec_per_head = d / VEC;
  const int lane = threadIdx.x & 31, sub = lane / LPR, sl = lane % LPR, wib = threadIdx.x >> 5;
  const int warps_total = (gridDim.x * blockDim.x) >> 5;
  const int warp_id = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  for (int64_t r0 = int64_t(win.row_begin) + int64_t(warp_id) * RPW; r0 < win.row_end;
       r0 += int64_t(warps_total) * RPW) {
    const int32_t row = int32_t(r0) + sub;
    const bool live = row < win.row_end;
    if (live) {
      const T* z = Z + size_t(row - win.win_base) * H;
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const int vi = v * LPR + sl;
        if (vi < NV) {
          float f[VEC];
          load_vec(z + vi * VEC, f);
          float ps = 0.f, pd = 0.f;
#pragma unroll
          for (int t = 0; t < VEC; ++t) {
            ps = fmaf(f[t], __ldg(a_src + vi * VEC + t), ps);
            pd = fmaf(f[t], __ldg(a_dst + vi * VEC + t), pd);
          }
          part[wib][sub][vi][0] = ps;
          part[wib][sub][vi][1] = pd;
        }
      }
    }
    __syncwarp();
    if (live) {
      for (int k = sl; k < K; k += LPR) {
        float ss = 0.f, sd = 0.f;
        for (int v = k * vec_per_head; v < (k + 1) * vec_per_head; ++v) {
          ss += part[wib][sub][v][0];
          sd += part[wib][sub][v][1];
        }
        scores[size_t(row - win.win_base) * K + k] = make_float2(ss * kLog2e, sd * kLog2e);
      }
    }
    __syncwarp();
  }
}

// ---- Eq. 7: edge scores, softmax over producers + self, weighted sum of Z rows, bias, ReLU ---
// A warp takes blocks of 32 consecutive destination rows: row pointers and producer ids of the
// whole block are fetched with a few coalesced loads into shared memory, so that the per-row work
// starts straight at the gathers of Z.  The half-scores arrive already multiplied by log2(e)
// (LeakyReLU commutes with a positive factor), so the softmax weights are plain exp2.  Producers
// are taken in groups of up to four: all their loads are issued first, the running maximum is
// updated once per group and the partial sum rescaled only if it grew.  Every Z row and every
// score is read once.
constexpr int kAggBlockRows = 32;
constexpr int kAggColCap = 224;       // producer ids cached per block of rows

__device__ __forceinline__ float lrelu(float x) { return fmaxf(x, 0.2f * x); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One group of NB (1..4) producers of a row: loads, then maximum, weights, accumulation.
template <typename T, int NB>
__device__ __forceinline__ void agg_group(const int32_t* __restrict__ js, int32_t win_base,
                                          const T* __restrict__ zlane, const float2* __restrict__ slane,
                                          int H, int K, float sd, float& m, float& l,
                                          float (&acc)[VecOf<T>::N]) {
  constexpr int VEC = VecOf<T>::N;
  float ev[NB];
  uint4 raw[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const int32_t j = js[b] - win_base;
    ev[b] = __ldg(&slane[size_t(j) * K].x);
    raw[b] = __ldg(reinterpret_cast<const uint4*>(zlane + size_t(j) * H));
  }
  float mx = m;
#pragma unroll
  for (int b = 0; b < NB; ++b) { ev[b] = lrelu(ev[b] + sd); mx = fmaxf(mx, ev[b]); }
  if (mx > m) {
    const float scale = fast_exp2(m - mx);
    l *= scale;
#pragma unroll
    for (int t = 0; t < VEC; ++t) acc[t] *= scale;
    m = mx;
  }
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const float p = fast_exp2(ev[b] - m);
    l += p;
    float z[VEC];
    unpack(raw[b], z);
#pragma unroll
    for (int t = 0; t < VEC; ++t) acc[t] = fmaf(p, z[t], acc[t]);
  }
}

template <typename T, int LPR, int VPL>
__global__ void __launch_bounds__(kRowThreads, (VPL == 1 ? 4 : 2))
k_aggregate(const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
            const T* __restrict__ Z, const float2* __restrict__ scores,
            const float* __restrict__ bias, T* __restrict__ h_out, int H, int K, Window win,
            const int32_t* __restrict__ self_idx, int block_rows) {
  constexpr int VEC = VecOf<T>::N;
  constexpr int RPW = 32 / LPR;
  constexpr int WARPS = kRowThreads / 32;
  __shared__ int32_t s_rp[WARPS][kAggBlockRows + 1];
  __shared__ int32_t s_col[WARPS][kAggColCap];
  const int NV = H / VEC, d = H / K;
  const int lane = threadIdx.x & 31, sub = lane / LPR, sl = lane % LPR, wib = threadIdx.x >> 5;
  const int warps_total = (gridDim.x * blockDim.x) >> 5;
  const int warp_id = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;

  int c0[VPL], head[VPL];
  bool on[VPL];
  float bs[VPL][VEC];
#pragma unroll
  for (int v = 0; v < VPL; ++v) {
    const int vi = v * LPR + sl;
    on[v] = vi < NV;
    c0[v] = on[v] ? vi * VEC : 0;
    head[v] = c0[v] / d;
#pragma unroll
    for (int t = 0; t < VEC; ++t) bs[v][t] = __ldg(bias + c0[v] + t);
  }

  // blocks of rows: as many rows (up to 32) as keep the block's producer ids within the cache;
  // a single row with more producers than that is walked straight from global memory
  // block_rows <= kAggBlockRows rows per warp and pass: fewer when the batch is small, so that every
  // warp of the grid has work
  int64_t r0 = int64_t(win.row_begin) + int64_t(warp_id) * block_rows;
  while (r0 < win.row_end) {
    const int nr = int(min(int64_t(block_rows), win.row_end - r0));
    __syncwarp();                                   // the previous block's reads are done
    if (lane < nr) s_rp[wib][lane] = __ldg(rowptr + r0 + lane);
    if (lane == 0) s_rp[wib][nr] = __ldg(rowptr + r0 + nr);
    __syncwarp();
    const int32_t eb = s_rp[wib][0];
    const int ne = min(s_rp[wib][nr] - eb, kAggColCap);
    for (int t = lane; t < ne; t += 32) s_col[wib][t] = __ldg(col + eb + t);
    __syncwarp();

    for (int rr = sub; rr < nr; rr += RPW) {
      const int32_t lrow = int32_t(r0) + rr - win.win_base;
      const int e0 = s_rp[wib][rr] - eb;              // edge offsets relative to the block
      const int n = s_rp[wib][rr + 1] - eb - e0;
      const bool cached = e0 + n <= kAggColCap;
      const int32_t* js = cached ? &s_col[wib][e0] : col + eb + e0;
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        if (!on[v]) continue;
        const T* zlane = Z + c0[v];
        const float2* slane = scores + head[v];
        const int32_t srow = self_idx ? __ldg(self_idx + int32_t(r0) + rr) : lrow;   // where the row's own Z lives
        const float2 self = __ldg(slane + size_t(srow) * K);
        const float sd = self.y;
        float m = lrelu(self.x + sd);                               // the self term opens the softmax
        float l = 1.f, acc[VEC];
        load_vec(zlane + size_t(srow) * H, acc);
        int t = 0;
        for (; t + 4 <= n; t += 4) agg_group<T, 4>(js + t, win.win_base, zlane, slane, H, K, sd, m, l, acc);
        const int rem = n - t;                          // the same for all lanes of a row group
        if (rem == 1) agg_group<T, 1>(js + t, win.win_base, zlane, slane, H, K, sd, m, l, acc);
        else if (rem == 2) agg_group<T, 2>(js + t, win.win_base, zlane, slane, H, K, sd, m, l, acc);
        else if (rem == 3) agg_group<T, 3>(js + t, win.win_base, zlane, slane, H, K, sd, m, l, acc);
        const float inv = __fdividef(1.f, l);
        float o[VEC];
#pragma unroll
        for (int t2 = 0; t2 < VEC; ++t2) o[t2] = fmaxf(fmaf(acc[t2], inv, bs[v][t2]), 0.f);
        store_vec(h_out + size_t(lrow) * H + c0[v], o);
      }
    }
    r0 += int64_t(warps_total) * block_rows;
  }
}

// ---- dispatch on the row geometry ------------------------------------------------------------
struct RowGeom { int lpr, vpl; };

template <typename T>
RowGeom row_geom(int H) {
  const int nv = H / VecOf<T>::N;
  if (nv <= 8) return {8, 1};
  if (nv == 16) return {16, 1};
  const int vpl = (nv + 31) / 32;
  return {32, vpl <= 1 ? 1 : (vpl == 2 ? 2 : 4)};
}

int row_grid(int64_t rows, int rpw) {
  const int64_t warps = (rows + rpw - 1) / rpw;
  const int64_t blocks = (warps + (kRowThreads / 32) - 1) / (kRowThreads / 32);
  const int64_t cap = int64_t(kNumSMs) * 8;
  return int(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

#define XRL_ROW_DISPATCH(TY_, H, CALL)                                         \
  do {                                                                       \
    const RowGeom g_ = row_geom<TY_>(H);                                       \
    if (g_.lpr == 8) { CALL(TY_, 8, 1); }                                      \
    else if (g_.lpr == 16) { CALL(TY_, 16, 1); }                               \
    else if (g_.vpl == 1) { CALL(TY_, 32, 1); }                                \
    else if (g_.vpl == 2) { CALL(TY_, 32, 2); }                                \
    else { CALL(TY_, 32, 4); }                                                 \
  } while (0)

}  // namespace

// one opt-in record per instantiation of k_embed (ensure_dynamic_smem keeps one flag array per kernel)
static int embed_slot(size_t elem, int lpr, int vpl) {
  return (elem == 2 ? 5 : 0) + (lpr == 8 ? 0 : lpr == 16 ? 1 : vpl == 1 ? 2 : vpl == 2 ? 3 : 4);
}

int launch_embed(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op,
                 const void* shape, const DevWeights& w, void* h, Window win, cudaStream_t st,
                 const int32_t* row_list, const void* eattr) {
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  if (rows <= 0) return 0;
  const size_t smem = sizeof(EmbedStage) * kEmbedWarps + sizeof(float) * size_t(2 * kS + 1) * d.H;
  static bool attr_set[10][64] = {};
#define CALL(TY_, LPR, VPL)                                                                        \
  if (smem > 48 * 1024 &&                                                                          \
      !ensure_dynamic_smem(k_embed<TY_, LPR, VPL>, int(smem), attr_set[embed_slot(sizeof(TY_), LPR, VPL)])) return -1; \
  k_embed<TY_, LPR, VPL><<<row_grid(rows, kEmbedRows), kRowThreads, smem, st>>>(                           \
      rowptr, col, op, static_cast<const TY_*>(shape), static_cast<const TY_*>(w.W0), w.b0,   \
      static_cast<TY_*>(h), d.H, d.T, win, row_list, static_cast<const TY_*>(eattr))
  if (d.dtype == XRL_BF16) XRL_ROW_DISPATCH(bf16, d.H, CALL);
  else XRL_ROW_DISPATCH(float, d.H, CALL);
#undef CALL
  return 1;
}

int launch_scores(const Dims& d, const void* Z, const LayerWeights& lw, float* scores, Window win,
                  cudaStream_t st) {
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  if (rows <= 0) return 0;
#define CALL(TY_, LPR, VPL)                                                                        \
  k_scores<TY_, LPR, VPL><<<row_grid(rows, 32 / LPR), kRowThreads, 0, st>>>(                       \
      static_cast<const TY_*>(Z), lw.a_src, lw.a_dst, reinterpret_cast<float2*>(scores), d.H, d.K, win)
  if (d.dtype == XRL_BF16) XRL_ROW_DISPATCH(bf16, d.H, CALL);
  else XRL_ROW_DISPATCH(float, d.H, CALL);
#undef CALL
  return 1;
}

int launch_aggregate(const Dims& d, const int32_t* rowptr, const int32_t* col, const void* Z,
                     const float* scores, const float* bias, void* h_out,
                     Window win, int64_t buf_rows, int32_t* status, cudaStream_t st,
                     const int32_t* self_idx) {
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  if (rows <= 0) return 0;
  {   // 512-byte rows with 4 | K: gathers by the TMA engine
    const int k = launch_aggregate_tma(d, rowptr, col, Z, scores, bias, h_out, win, buf_rows, nullptr, nullptr, status, st,
                                       self_idx);
    if (k >= 0 || d.zmerged) return k;       // with merged rows there is no other kernel to fall back to
  }
  // rows per warp and pass: the 32 of a full block, fewer for small batches (a multiple of the rows a
  // warp holds at once)
  const int64_t warps_avail = int64_t(kNumSMs) * 8 * (kRowThreads / 32);
#define CALL(TY_, LPR, VPL)                                                                        \
  do {                                                                                             \
    const int rpw_ = 32 / LPR;                                                                     \
    int64_t br_ = (rows + warps_avail - 1) / warps_avail;                                          \
    br_ = ((br_ + rpw_ - 1) / rpw_) * rpw_;                                                        \
    if (br_ > kAggBlockRows) br_ = kAggBlockRows;                                                  \
    k_aggregate<TY_, LPR, VPL><<<row_grid(rows, int(br_)), kRowThreads, 0, st>>>(                  \
        rowptr, col, static_cast<const TY_*>(Z), reinterpret_cast<const float2*>(scores), bias,    \
        static_cast<TY_*>(h_out), d.H, d.K, win, self_idx, int(br_));                              \
  } while (0)
  if (d.dtype == XRL_BF16) XRL_ROW_DISPATCH(bf16, d.H, CALL);
  else XRL_ROW_DISPATCH(float, d.H, CALL);
#undef CALL
  return 1;
}

}  // namespace xrl

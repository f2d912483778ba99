// Per-graph readout and global update (paper Eq. 8), the policy and value heads with
// invalid-action masking and No-Op (Sections 3.3.2, 3.3.3), and the categorical draw.
// Every reduction runs in a fixed order (no floating-point atomics), so results are
// reproducible run to run.
#include "xrl_internal.cuh"

namespace xrl {

namespace {

constexpr int kRoThreads = 256;

// sum_k x[k] * W[k * ld + c]: the weight loads are issued DEPTH (then eight) at a time so that their
// latencies overlap; the additions keep the order k = 0, 1, 2, ...  DEPTH = 32 is for launches of few
// CTAs, which are bound by the latency of these loads; with many CTAs per SM the registers it takes cost
// more occupancy than the depth gains, and DEPTH = 8 is used.
template <int DEPTH>
__device__ __forceinline__ float column_dot(const float* x, int in, const float* __restrict__ W, int ld,
                                            int c, float acc) {
  int k = 0;
  if (DEPTH > 8) {
    for (; k + DEPTH <= in; k += DEPTH) {
      float w[DEPTH];
#pragma unroll
      for (int t = 0; t < DEPTH; ++t) w[t] = __ldg(W + size_t(k + t) * ld + c);
#pragma unroll
      for (int t = 0; t < DEPTH; ++t) acc = fmaf(x[k + t], w[t], acc);
    }
  }
  for (; k + 8 <= in; k += 8) {
    float w[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) w[t] = __ldg(W + size_t(k + t) * ld + c);
#pragma unroll
    for (int t = 0; t < 8; ++t) acc = fmaf(x[k + t], w[t], acc);
  }
  for (; k < in; ++k) acc = fmaf(x[k], __ldg(W + size_t(k) * ld + c), acc);
  return acc;
}

// y[c] = bias[c] + sum_k x[k] W[k * ld + c] for c < ncols, for every thread block shape: with fewer columns
// than threads the k range is cut into P = blockDim / CP contiguous parts (CP = columns per pass, a power of
// two), the parts are computed by different thread groups and added in part order.  Every thread of the
// block calls it; `part` is blockDim floats of scratch; emit(c, y) runs once per column.
template <int DEPTH, typename Emit>
__device__ __forceinline__ void dense_columns(const float* x, int in, const float* __restrict__ W, int ld,
                                              int ncols, const float* __restrict__ bias, float* part, Emit emit) {
  const int nt = blockDim.x, tid = threadIdx.x;
  int CP = 32;
  while (CP < ncols && CP < nt) CP <<= 1;
  const int P = nt / CP, cl = tid % CP, p = tid / CP;
  if (P == 1) {                                  // as many columns as threads (or more): no split, no barriers
    for (int c = tid; c < ncols; c += nt) emit(c, column_dot<DEPTH>(x, in, W, ld, c, bias[c]));
    return;
  }
  const int k0 = int((int64_t(in) * p) / P), k1 = int((int64_t(in) * (p + 1)) / P);
  for (int c0 = 0; c0 < ncols; c0 += CP) {
    const int c = c0 + cl;
    part[tid] = (c < ncols) ? column_dot<DEPTH>(x + k0, k1 - k0, W + size_t(k0) * ld, ld, c, 0.f) : 0.f;
    __syncthreads();
    if (p == 0 && c < ncols) {
      float y = bias[c];
      for (int q = 0; q < P; ++q) y += part[q * CP + cl];
      emit(c, y);
    }
    __syncthreads();
  }
}

// ---- readout, stage 1: column sums of one chunk of consecutive rows of one graph -------------
template <typename T>
__global__ void __launch_bounds__(kRoThreads)
k_readout(const T* __restrict__ h, const int32_t* __restrict__ chunk_row0,
          const int32_t* __restrict__ chunk_row1, int32_t chunk_begin, float* __restrict__ partial,
          int H, int32_t win_base, const int32_t* __restrict__ remap) {
  constexpr int VEC = VecOf<T>::N;
  extern __shared__ float red[];                 // [RG][H]
  const int NV = H / VEC;
  const int RG = kRoThreads / NV;                // row groups working in parallel
  const int32_t chunk = chunk_begin + blockIdx.x;
  const int32_t r0 = chunk_row0[chunk], r1 = chunk_row1[chunk];
  const int vi = threadIdx.x % NV, rg = threadIdx.x / NV;
  float acc[VEC];
#pragma unroll
  for (int t = 0; t < VEC; ++t) acc[t] = 0.f;
  if (rg < RG) {
    int32_t r = r0 + rg;
    for (; r + 3 * RG < r1; r += 4 * RG) {
      float f[4][VEC];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        load_vec(h + size_t(remap ? __ldg(remap + r + u * RG) : r + u * RG - win_base) * H + vi * VEC, f[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int t = 0; t < VEC; ++t) acc[t] += f[u][t];
    }
    for (; r < r1; r += RG) {
      float f[VEC];
      load_vec(h + size_t(remap ? __ldg(remap + r) : r - win_base) * H + vi * VEC, f);
#pragma unroll
      for (int t = 0; t < VEC; ++t) acc[t] += f[t];
    }
#pragma unroll
    for (int t = 0; t < VEC; ++t) red[rg * H + vi * VEC + t] = acc[t];
  }
  __syncthreads();
  for (int c = threadIdx.x; c < H; c += kRoThreads) {
    float s = 0.f;
    for (int g = 0; g < RG; ++g) s += red[g * H + c];
    partial[size_t(chunk) * H + c] = s;
  }
}

// ---- Eq. 8: emb_g = ReLU(Wg^T [ sum of the graph's chunk sums | g0_g ] + bg) -------------------
template <int DEPTH>
__global__ void __launch_bounds__(1024)
k_global_update(const float* __restrict__ partial, const int32_t* __restrict__ graph_chunk_off,
                const float* __restrict__ g0, const float* __restrict__ Wg,
                const float* __restrict__ bg, float* __restrict__ emb, int H, int Dg) {
  extern __shared__ float u[];                   // [H + Dg], then blockDim floats of scratch
  float* part = u + H + Dg;
  const int32_t g = blockIdx.x;
  const int32_t c0 = graph_chunk_off[g], c1 = graph_chunk_off[g + 1];
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    float s = 0.f;
    for (int32_t ch = c0; ch < c1; ++ch) s += partial[size_t(ch) * H + c];
    u[c] = s;
  }
  for (int t = threadIdx.x; t < Dg; t += blockDim.x) u[H + t] = g0 ? g0[size_t(g) * Dg + t] : 0.f;
  __syncthreads();
  dense_columns<DEPTH>(u, H + Dg, Wg, H, H, bg, part,
                [&](int c, float y) { emb[size_t(g) * H + c] = fmaxf(y, 0.f); });
}

// Eq. 8 from the partial sums written by the aggregate kernel fused with the readout: per graph, the
// partial of the block in which the graph starts (if it does not start at the block's first row), then
// the partials of the following 32-row blocks whose first row belongs to the graph, in order.
template <int DEPTH>
__global__ void __launch_bounds__(1024)
k_global_update_blocks(const float* __restrict__ partial, const int32_t* __restrict__ node_off,
                       int32_t nblocks, int bshift, const float* __restrict__ g0, const float* __restrict__ Wg,
                       const float* __restrict__ bg, float* __restrict__ emb, int H, int Dg) {
  extern __shared__ __align__(16) float u[];     // [H + Dg], then (16-byte aligned) 4 blockDim floats of scratch
  float* part = u + ((H + Dg + 3) & ~3);
  const int32_t g = blockIdx.x;
  const int32_t start = node_off[g], end = node_off[g + 1];
  // With more threads than columns the blocks' partial sums are added in P interleaved parts (part p takes the
  // blocks b0 + p, b0 + p + P, ...), and the parts in order: a fixed order for a given launch shape.
  const int P = int(blockDim.x) >= 2 * H ? int(blockDim.x) / H : 1;
  if (P > 1 && (H & 3) == 0) {
    // four columns per thread (16-byte loads) and 4 P interleaved parts: with 1,024 threads and H = 256 a thread
    // adds every 16th block, so that a graph of 70 blocks costs one round of loads instead of five
    const int HV = H >> 2, PV = int(blockDim.x) / HV;
    const int cv = threadIdx.x % HV, p = threadIdx.x / HV;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    int32_t b0 = 0, b1 = -1;
    if (end > start) {
      b0 = start >> bshift;
      if (start & ((1 << bshift) - 1)) ++b0;
      b1 = (end - 1) >> bshift;
    }
    if (p < PV)
      for (int32_t b = b0 + p; b <= b1; b += PV) {
        const float4 v = *reinterpret_cast<const float4*>(partial + size_t(b) * H + 4 * cv);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
    if (p < PV) *reinterpret_cast<float4*>(part + size_t(p) * H + 4 * cv) = s;
    __syncthreads();
    if (int(threadIdx.x) < H) {
      const int c = threadIdx.x;
      float t = (end > start && (start & ((1 << bshift) - 1))) ? partial[size_t(nblocks + g) * H + c] : 0.f;
      for (int q = 0; q < PV; ++q) t += part[q * H + c];
      u[c] = t;
    }
  } else if (P == 1) {
    for (int c = threadIdx.x; c < H; c += blockDim.x) {
      float s = 0.f;
      if (end > start) {
        int32_t b0 = start >> bshift;
        if (start & ((1 << bshift) - 1)) { s += partial[size_t(nblocks + g) * H + c]; ++b0; }
        const int32_t b1 = (end - 1) >> bshift;
        for (int32_t b = b0; b <= b1; ++b) s += partial[size_t(b) * H + c];
      }
      u[c] = s;
    }
  } else {
    const int c = threadIdx.x % H, p = threadIdx.x / H;
    float s = 0.f;
    int32_t b0 = 0, b1 = -1;
    if (end > start) {
      b0 = start >> bshift;
      if (start & ((1 << bshift) - 1)) ++b0;
      b1 = (end - 1) >> bshift;
    }
    if (p < P)
      for (int32_t b = b0 + p; b <= b1; b += P) s += partial[size_t(b) * H + c];
    part[threadIdx.x] = s;
    __syncthreads();
    if (p == 0) {
      float t = (end > start && (start & ((1 << bshift) - 1))) ? partial[size_t(nblocks + g) * H + c] : 0.f;
      for (int q = 0; q < P; ++q) t += part[q * H + c];
      u[c] = t;
    }
  }
  for (int t = threadIdx.x; t < Dg; t += blockDim.x) u[H + t] = g0 ? g0[size_t(g) * Dg + t] : 0.f;
  __syncthreads();
  dense_columns<DEPTH>(u, H + Dg, Wg, H, H, bg, part,
                [&](int c, float y) { emb[size_t(g) * H + c] = fmaxf(y, 0.f); });
}

// Block-wide sum in a fixed order (lanes of a warp by a shuffle tree, then the warps' sums by one warp's
// shuffle tree): the same for the same blockDim, two barriers.  Every thread contributes v and gets the sum;
// `scratch` holds at least 32 floats.  blockDim is a multiple of 32.
__device__ float block_sum(float v, float* scratch) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if (lane == 0) scratch[wid] = v;
  __syncthreads();
  float r = lane < nw ? scratch[lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xFFFFFFFFu, r, o);
  __syncthreads();
  return r;
}
__device__ float block_max(float v, float* scratch) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  if (lane == 0) scratch[wid] = v;
  __syncthreads();
  float r = lane < nw ? scratch[lane] : -INFINITY;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xFFFFFFFFu, r, o));
  __syncthreads();
  return r;
}

// A head's MLP (Section 3.3.2): out = w2 . ReLU(W1^T x + b1) + b2, or with a second hidden width hid2 > 0
// out = w2 . ReLU(Wh^T ReLU(W1^T x + b1) + bh) + b2.  x (length `in`) and y1 (hid floats, used only when
// hid2 > 0) are in shared memory; all threads return the result.
struct Mlp { const float *W1, *b1, *Wh, *bh, *w2, *b2; int hid, hid2; };
template <int DEPTH>
__device__ float mlp_scalar(const float* x, int in, const Mlp& m, float* y1, float* scratch) {
  float contrib = 0.f;
  if (m.hid2 <= 0) {
    dense_columns<DEPTH>(x, in, m.W1, m.hid, m.hid, m.b1, scratch, [&](int c, float y) { contrib += fmaxf(y, 0.f) * m.w2[c]; });
  } else {
    dense_columns<DEPTH>(x, in, m.W1, m.hid, m.hid, m.b1, scratch, [&](int c, float y) { y1[c] = fmaxf(y, 0.f); });
    __syncthreads();
    dense_columns<DEPTH>(y1, m.hid, m.Wh, m.hid2, m.hid2, m.bh, scratch,
                  [&](int c, float y) { contrib += fmaxf(y, 0.f) * m.w2[c]; });
  }
  return block_sum(contrib, scratch) + m.b2[0];
}

// ---- policy MLP: one scalar score per graph -----------------------------------------------------
template <int DEPTH>
__global__ void __launch_bounds__(1024)
k_policy_logit(const float* __restrict__ emb, const Mlp mlp, float* __restrict__ logit, int H) {
  extern __shared__ float sm[];                  // [H] + [blockDim] + [hid]
  float* x = sm;
  float* scratch = sm + H;
  float* y1 = scratch + blockDim.x;
  const int32_t g = blockIdx.x;
  for (int c = threadIdx.x; c < H; c += blockDim.x) x[c] = emb[size_t(g) * H + c];
  __syncthreads();
  const float v = mlp_scalar<DEPTH>(x, H, mlp, y1, scratch);
  if (threadIdx.x == 0) logit[g] = v;
}

// The rest of a head's MLP behind its first layer: y1 = ReLU(W1^T x + b1) is given (hid floats in shared
// memory); all threads return the result.
template <int DEPTH>
__device__ float mlp_tail(const float* y1, const Mlp& m, float* scratch) {
  float contrib = 0.f;
  if (m.hid2 <= 0) {
    for (int c = threadIdx.x; c < m.hid; c += blockDim.x) contrib += y1[c] * m.w2[c];
  } else {
    dense_columns<DEPTH>(y1, m.hid, m.Wh, m.hid2, m.hid2, m.bh, scratch,
                  [&](int c, float y) { contrib += fmaxf(y, 0.f) * m.w2[c]; });
  }
  return block_sum(contrib, scratch) + m.b2[0];
}

// ---- steps of few graphs and environments: policy scores and the value head's first layer in one launch ------
// CTAs [0, B) are k_policy_logit.  CTAs B + e * VC + ch compute chunk ch (hid / VC columns) of the value head's
// first layer for environment e: y1[e] = ReLU(W1^T [emb(current) | mean of the valid candidates' emb] + b1), the
// candidate mean taken inside the CTA (part p of the threads adds candidates p, p + P, ... in order, the parts
// in order).  The 2H x hid weights are then read by VC CTAs instead of by the one CTA of the environment.
template <int DEPTH>
__global__ void __launch_bounds__(1024)
k_policy_value_hidden(const float* __restrict__ emb, const Mlp pm, float* __restrict__ logit, int H, int32_t B,
                      const int32_t* __restrict__ env_off, const uint8_t* __restrict__ mask, int A, const Mlp vm,
                      float* __restrict__ y1v, int VC) {
  extern __shared__ float sm[];                  // policy: [H] + [blockDim] + [hid]; value: [2H] + [blockDim]
  const int nt = blockDim.x, tid = threadIdx.x;
  if (int32_t(blockIdx.x) < B) {
    float* x = sm;
    float* scratch = sm + H;
    float* y1 = scratch + nt;
    const int32_t g = blockIdx.x;
    for (int c = tid; c < H; c += nt) x[c] = emb[size_t(g) * H + c];
    __syncthreads();
    const float v = mlp_scalar<DEPTH>(x, H, pm, y1, scratch);
    if (tid == 0) logit[g] = v;
    return;
  }
  float* u = sm;                                 // [2H]
  float* scratch = sm + 2 * H;                   // [blockDim]
  const int32_t e = (int32_t(blockIdx.x) - B) / VC, ch = (int32_t(blockIdx.x) - B) % VC;
  const int32_t cur = env_off[e];
  const int32_t C = env_off[e + 1] - cur - 1;
  const uint8_t* mk = mask + size_t(e) * A;
  float cnt = 0.f;
  for (int a = tid; a < C && a < A; a += nt) cnt += mk[a] ? 1.f : 0.f;
  const float nv = block_sum(cnt, scratch);
  const int P = nt >= 2 * H ? nt / H : 1;
  {
    const int c = tid % H, p = tid / H;
    float s = 0.f;
    if (p < P && tid < P * H)
      for (int a = p; a < C && a < A; a += P)
        if (mk[a]) s += emb[size_t(cur + 1 + a) * H + c];
    scratch[tid] = s;
    __syncthreads();
    if (tid < H) {
      float t = 0.f;
      for (int q = 0; q < P; ++q) t += scratch[q * H + tid];
      u[tid] = emb[size_t(cur) * H + tid];
      u[H + tid] = nv > 0.f ? t / nv : 0.f;
    }
    __syncthreads();
  }
  const int CW = (vm.hid + VC - 1) / VC, c_lo = ch * CW, ncols = min(CW, vm.hid - c_lo);
  if (ncols > 0)
    dense_columns<DEPTH>(u, 2 * H, vm.W1 + c_lo, vm.hid, ncols, vm.b1 + c_lo, scratch,
                  [&](int c, float y) { y1v[size_t(e) * vm.hid + c_lo + c] = fmaxf(y, 0.f); });
}

// ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) -----------------------------------------
struct U4 { uint32_t x, y, z, w; };
__device__ U4 philox4x32_10(uint32_t k0, uint32_t k1, U4 c) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t lo0 = 0xD2511F53u * c.x, hi0 = __umulhi(0xD2511F53u, c.x);
    const uint32_t lo1 = 0xCD9E8D57u * c.z, hi1 = __umulhi(0xCD9E8D57u, c.z);
    c = U4{hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0};
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

__device__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* scratch) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  if (lane == 0) scratch[wid] = v;
  __syncthreads();
  unsigned long long r = lane < nw ? scratch[lane] : 0ull;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xFFFFFFFFu, r, o);
  __syncthreads();
  return r;
}

// Categorical draw from fp32 probabilities p[0..A1) with integer arithmetic only.
// scratch: blockDim.x + 1 unsigned 64-bit words.  Every thread returns the action.
__device__ int32_t sample_row(const float* __restrict__ p, int A1, uint64_t seed, uint64_t step,
                              uint32_t env, unsigned long long* scratch) {
  const int tid = threadIdx.x, nt = blockDim.x;
  // contiguous slice per thread so that prefix order = index order
  const int per = (A1 + nt - 1) / nt;
  const int a0 = min(A1, tid * per), a1 = min(A1, a0 + per);
  unsigned long long mine = 0;
  for (int a = a0; a < a1; ++a) mine += (unsigned long long)floorf(p[a] * 4294967296.0f);
  const unsigned long long Q = block_sum_u64(mine, scratch);
  if (Q == 0) return A1 - 1;
  const U4 r = philox4x32_10(uint32_t(seed), uint32_t(seed >> 32),
                             U4{env, uint32_t(step), uint32_t(step >> 32), 0u});
  const unsigned long long r64 = (unsigned long long)r.x | ((unsigned long long)r.y << 32);
  const unsigned long long t = __umul64hi(r64, Q);
  // exclusive prefix of the per-thread totals: scan inside each warp, then over the warp totals
  // (integer sums: any association gives the same result)
  {
    const int lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += y;
    }
    __syncthreads();                            // scratch is free again after block_sum_u64
    if (lane == 31) scratch[wid] = incl;
    __syncthreads();
    unsigned long long wbase = 0;
    for (int w = 0; w < wid && w < nw; ++w) wbase += scratch[w];
    __syncthreads();
    scratch[tid] = wbase + incl - mine;
    if (tid == 0) scratch[nt] = (unsigned long long)(A1 - 1);
  }
  __syncthreads();
  unsigned long long run = scratch[tid];
  if (run <= t && t < run + mine) {              // exactly one thread owns t
    for (int a = a0; a < a1; ++a) {
      run += (unsigned long long)floorf(p[a] * 4294967296.0f);
      if (run > t) { scratch[nt] = (unsigned long long)a; break; }
    }
  }
  __syncthreads();
  const int32_t act = int32_t(scratch[nt]);
  __syncthreads();
  return act;
}

// ---- sum of the valid candidates' embeddings of one environment, 32 columns per CTA ---------------
// 1024 threads = 32 columns x 32 parts; part p adds candidates p, p + 32, ... in order, the parts are
// then added in order: a fixed summation order, so the result is reproducible.
__global__ void __launch_bounds__(1024)
k_candidate_sum(const float* __restrict__ emb, const int32_t* __restrict__ env_off,
                const uint8_t* __restrict__ mask, float* __restrict__ cand_sum, int H, int A) {
  __shared__ float part[32][33];
  const int32_t e = blockIdx.x;
  const int c = blockIdx.y * 32 + (threadIdx.x & 31), p = threadIdx.x >> 5;
  const int32_t cur = env_off[e];
  const int32_t C = env_off[e + 1] - cur - 1;
  const uint8_t* mk = mask + size_t(e) * A;
  float s = 0.f;
  if (c < H)
    for (int a = p; a < C; a += 32)
      if (mk[a]) s += emb[size_t(cur + 1 + a) * H + c];
  part[p][threadIdx.x & 31] = s;
  __syncthreads();
  if (p == 0 && c < H) {
    float t = 0.f;
    for (int q = 0; q < 32; ++q) t += part[q][threadIdx.x & 31];
    cand_sum[size_t(e) * H + c] = t;
  }
}

// ---- per environment: masked softmax, candidate mean, value MLP, optional draw -----------------
template <int DEPTH>
__global__ void __launch_bounds__(1024)
k_env_policy(const float* __restrict__ emb, const float* __restrict__ logit,
             const float* __restrict__ cand_sum,
             const int32_t* __restrict__ env_off, const uint8_t* __restrict__ mask,
             const Mlp vmlp, float* __restrict__ probs,
             float* __restrict__ value, int32_t* __restrict__ action, int H, int A,
             uint64_t seed, uint64_t step, int32_t* status, const float* __restrict__ y1_pre) {
  extern __shared__ unsigned long long sm64[];   // [nt + 1] u64, then floats
  const int nt = blockDim.x, tid = threadIdx.x;
  float* scratch = reinterpret_cast<float*>(sm64 + nt + 1);   // [nt]
  float* u = scratch + nt;                                    // [2H]
  float* y1 = u + 2 * H;                                      // [hid]
  const int32_t e = blockIdx.x;
  const int32_t cur = env_off[e];
  const int32_t C = env_off[e + 1] - cur - 1;
  const uint8_t* mk = mask + size_t(e) * A;
  float* pr = probs + size_t(e) * (A + 1);

  // masked softmax over the valid candidates and No-Op (index A, scored by the current graph)
  float mx = -INFINITY;
  for (int a = tid; a <= A; a += nt) {
    bool valid = (a == A);
    if (a < A && mk[a]) {
      if (a >= C) raise(status, XRL_ERR_INVALID_ARG); else valid = true;
    }
    if (valid) mx = fmaxf(mx, logit[a == A ? cur : cur + 1 + a]);
  }
  mx = block_max(mx, scratch);
  float se = 0.f;
  for (int a = tid; a <= A; a += nt) {
    const bool valid = (a == A) || (a < C && mk[a]);
    const float ex = valid ? expf(logit[a == A ? cur : cur + 1 + a] - mx) : 0.f;
    pr[a] = ex;
    se += ex;
  }
  const float denom = block_sum(se, scratch);
  for (int a = tid; a <= A; a += nt) pr[a] = pr[a] / denom;     // each thread rewrites its own entries

  float v;
  if (y1_pre != nullptr) {
    // the value head's first layer was computed by k_policy_value_hidden: the rest of the MLP
    for (int c = tid; c < vmlp.hid; c += nt) y1[c] = y1_pre[size_t(e) * vmlp.hid + c];
    __syncthreads();
    v = mlp_tail<DEPTH>(y1, vmlp, scratch);
  } else {
    // value head input: [ emb(current) | mean of emb over the valid candidates ]
    for (int c = tid; c < H; c += nt) u[c] = emb[size_t(cur) * H + c];
    float cnt = 0.f;
    for (int a = tid; a < C; a += nt) cnt += mk[a] ? 1.f : 0.f;
    const float nv = block_sum(cnt, scratch);
    for (int c = tid; c < H; c += nt) u[H + c] = nv > 0.f ? cand_sum[size_t(e) * H + c] / nv : 0.f;
    __syncthreads();
    v = mlp_scalar<DEPTH>(u, 2 * H, vmlp, y1, scratch);
  }
  if (tid == 0) value[e] = v;

  if (action != nullptr) {
    __syncthreads();                              // probs of this row are written by this block
    const int32_t act = sample_row(pr, A + 1, seed, step, uint32_t(e), sm64);
    if (tid == 0) action[e] = act;
  }
}

__global__ void __launch_bounds__(1024)
k_sample(const float* __restrict__ probs, int A1, uint64_t seed, uint64_t step,
         int32_t* __restrict__ action) {
  extern __shared__ unsigned long long sm64[];
  const int32_t e = blockIdx.x;
  const int32_t act = sample_row(probs + size_t(e) * A1, A1, seed, step, uint32_t(e), sm64);
  if (threadIdx.x == 0) action[e] = act;
}

// Seeded initial weights: element i of the blob is bound * u_i, u_i = (w >> 8) * 2^-23 - 1 in [-1, 1) with w the
// first word of Philox4x32-10(key = seed, counter = (i, 0, 0, 1)); every step is exact in fp32 except the one
// product, so any IEEE implementation gives the same bits.  (Counter word 3 = 1 keeps this stream apart from
// the action draws, which use 0.)
__global__ void k_init_weights(float* __restrict__ blob, int64_t first, int64_t count, float bound, uint32_t k0,
                               uint32_t k1) {
  const int64_t t = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= count) return;
  const uint64_t i = uint64_t(first + t);
  const U4 r = philox4x32_10(k0, k1, U4{uint32_t(i), uint32_t(i >> 32), 0u, 1u});
  const float u = __fsub_rn(__fmul_rn(float(r.x >> 8), 1.1920928955078125e-07f), 1.0f);
  blob[first + t] = __fmul_rn(bound, u);
}

__global__ void k_to_float_bf16(const bf16* __restrict__ src, float* __restrict__ dst, int64_t n) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = __bfloat162float(src[i]);
}

// dst = storage-type copy of src [rows x cols]; dst_t (optional) = its transpose [cols x rows]
template <typename T>
__global__ void k_round_weights(const float* __restrict__ src, T* __restrict__ dst,
                                T* __restrict__ dst_t, int rows, int cols) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * cols) return;
  const int r = i / cols, c = i - r * cols;
  const T v = T(src[i]);
  dst[i] = v;
  if (dst_t != nullptr) dst_t[size_t(c) * rows + r] = v;
}

// Launches with at most a few CTAs per SM are bound by the latency of their weight loads.
bool few_ctas(int64_t ctas) { return ctas <= 4 * kNumSMs; }
// With fewer CTAs than SMs every CTA has an SM to itself and the chain of dependent weight loads of one thread
// is the whole run time: 1,024 threads cut every column's sum into four parts (dense_columns) instead of one.
int head_threads(int64_t ctas) { return ctas <= kNumSMs ? 1024 : 256; }

int pow2_threads(int want) {          // power of two in [32, 1024] (block_sum needs a power of two)
  int t = 32;
  while (t < want && t < 1024) t <<= 1;
  return t;
}

}  // namespace

int launch_readout(const Dims& d, const void* h, const int32_t* chunk_row0, const int32_t* chunk_row1,
                   int32_t chunk_begin, int32_t chunk_end, float* partial, int32_t win_base,
                   cudaStream_t st, const int32_t* remap) {
  const int n = chunk_end - chunk_begin;
  if (n <= 0) return 0;
  if (d.dtype == XRL_BF16) {
    const int RG = kRoThreads / (d.H / 8);
    k_readout<bf16><<<n, kRoThreads, sizeof(float) * size_t(RG) * d.H, st>>>(
        static_cast<const bf16*>(h), chunk_row0, chunk_row1, chunk_begin, partial, d.H, win_base, remap);
  } else {
    const int RG = kRoThreads / (d.H / 4);
    k_readout<float><<<n, kRoThreads, sizeof(float) * size_t(RG) * d.H, st>>>(
        static_cast<const float*>(h), chunk_row0, chunk_row1, chunk_begin, partial, d.H, win_base, remap);
  }
  return 1;
}

int launch_global_update(const Dims& d, const float* partial, const int32_t* graph_chunk_off,
                         const float* g0, const DevWeights& w, float* emb, int32_t B, cudaStream_t st) {
  if (B <= 0) return 0;
  const int nt = head_threads(B);
  const size_t smem = sizeof(float) * size_t(d.H + d.Dg + nt);
  if (few_ctas(B)) k_global_update<32><<<B, nt, smem, st>>>(partial, graph_chunk_off, g0, w.Wg, w.bg, emb, d.H, d.Dg);
  else k_global_update<8><<<B, nt, smem, st>>>(partial, graph_chunk_off, g0, w.Wg, w.bg, emb, d.H, d.Dg);
  return 1;
}

int launch_global_update_blocks(const Dims& d, const float* partial, const int32_t* node_off, int32_t nblocks,
                                int block_shift, const float* g0, const DevWeights& w, float* emb, int32_t B,
                                cudaStream_t st) {
  if (B <= 0) return 0;
  const int nt = head_threads(B);
  const size_t smem = sizeof(float) * size_t(d.H + d.Dg + 3 + 4 * nt);   // the block sums' parts take 4 floats per thread
  if (few_ctas(B))
    k_global_update_blocks<32><<<B, nt, smem, st>>>(partial, node_off, nblocks, block_shift, g0, w.Wg, w.bg, emb, d.H, d.Dg);
  else
    k_global_update_blocks<8><<<B, nt, smem, st>>>(partial, node_off, nblocks, block_shift, g0, w.Wg, w.bg, emb, d.H, d.Dg);
  return 1;
}

int launch_heads(const Dims& d, const DevWeights& w, const float* emb, const int32_t* env_off,
                 const uint8_t* mask, int32_t B, int32_t num_envs, float* logit_ws, float* probs,
                 float* value, int32_t* action, uint64_t seed, uint64_t step, int32_t* status,
                 cudaStream_t st) {
  if (B <= 0 || num_envs <= 0) return 0;
  const Mlp pm{w.pW1, w.pb1, w.pWh, w.pbh, w.pw2, w.pb2, d.Hm, d.Hm2};
  const Mlp vm{w.vW1, w.vb1, w.vWh, w.vbh, w.vw2, w.vb2, d.Hm, d.Hm2};
  float* cand_sum = logit_ws + B;                 // [num_envs x H], behind the per-graph logits
  // Steps of few graphs and environments with a short action space (the paper's own sizes): two launches, the
  // value head's first layer spread over kValueChunks CTAs per environment next to the policy CTAs.
  constexpr int kValueChunks = 8;
  if (B + num_envs * kValueChunks <= kNumSMs && d.A <= 256 && d.Hm <= d.H) {
    const int nt = 1024;
    const size_t sm1 = sizeof(float) * size_t(2 * d.H + nt + d.Hm);
    float* y1v = cand_sum;                        // [num_envs x Hm] (Hm <= H): the candidate sums are not needed here
    k_policy_value_hidden<32><<<B + num_envs * kValueChunks, nt, sm1, st>>>(emb, pm, logit_ws, d.H, B, env_off, mask,
                                                                         d.A, vm, y1v, kValueChunks);
    const size_t smem = sizeof(unsigned long long) * size_t(nt + 1) + sizeof(float) * size_t(nt + 2 * d.H + d.Hm);
    k_env_policy<32><<<num_envs, nt, smem, st>>>(emb, logit_ws, cand_sum, env_off, mask, vm, probs, value, action,
                                                 d.H, d.A, seed, step, status, y1v);
    return 2;
  }
  const int pnt = head_threads(B);
  const size_t psm = sizeof(float) * size_t(d.H + pnt + d.Hm);
  if (few_ctas(B)) k_policy_logit<32><<<B, pnt, psm, st>>>(emb, pm, logit_ws, d.H);
  else k_policy_logit<8><<<B, pnt, psm, st>>>(emb, pm, logit_ws, d.H);
  k_candidate_sum<<<dim3(num_envs, (d.H + 31) / 32), 1024, 0, st>>>(emb, env_off, mask, cand_sum, d.H, d.A);
  int want = d.H > d.A + 1 ? d.H : d.A + 1;
  if (want < 256) want = 256;               // enough threads to split the value head's dense map
  if (num_envs <= kNumSMs) want = 1024;     // (an SM per environment: see head_threads)
  const int nt = pow2_threads(want);
  const size_t smem = sizeof(unsigned long long) * size_t(nt + 1) + sizeof(float) * size_t(nt + 2 * d.H + d.Hm);
  if (few_ctas(num_envs))
    k_env_policy<32><<<num_envs, nt, smem, st>>>(emb, logit_ws, cand_sum, env_off, mask, vm, probs, value, action,
                                                 d.H, d.A, seed, step, status, nullptr);
  else
    k_env_policy<8><<<num_envs, nt, smem, st>>>(emb, logit_ws, cand_sum, env_off, mask, vm, probs, value, action,
                                                d.H, d.A, seed, step, status, nullptr);
  return 3;
}

int launch_sample(const float* probs, int32_t num_envs, int32_t A1, uint64_t seed, uint64_t step,
                  int32_t* action, cudaStream_t st) {
  if (num_envs <= 0) return 0;
  const int nt = pow2_threads(A1);
  k_sample<<<num_envs, nt, sizeof(unsigned long long) * size_t(nt + 1), st>>>(probs, A1, seed, step,
                                                                              action);
  return 1;
}

int launch_init_weights(float* blob, int64_t first, int64_t count, float bound, uint64_t seed, cudaStream_t st) {
  if (count <= 0) return 0;
  k_init_weights<<<unsigned((count + 255) / 256), 256, 0, st>>>(blob, first, count, bound, uint32_t(seed),
                                                                uint32_t(seed >> 32));
  return 1;
}

int launch_to_float(const void* src, int dtype, float* dst, int64_t n, cudaStream_t st) {
  if (n <= 0) return 0;
  if (dtype == XRL_BF16) {
    k_to_float_bf16<<<unsigned((n + 255) / 256), 256, 0, st>>>(static_cast<const bf16*>(src), dst, n);
    return 1;
  }
  cudaMemcpyAsync(dst, src, sizeof(float) * size_t(n), cudaMemcpyDeviceToDevice, st);
  return 0;
}

int launch_round_weights(const float* src, void* dst, void* dst_t, int rows, int cols, int dtype,
                         cudaStream_t st) {
  const int n = rows * cols;
  if (dtype == XRL_BF16)
    k_round_weights<bf16><<<(n + 255) / 256, 256, 0, st>>>(src, static_cast<bf16*>(dst),
                                                          static_cast<bf16*>(dst_t), rows, cols);
  else
    k_round_weights<float><<<(n + 255) / 256, 256, 0, st>>>(src, static_cast<float*>(dst),
                                                           static_cast<float*>(dst_t), rows, cols);
  return 1;
}

}  // namespace xrl

// Reverse pass of the agent's forward path for the PPO objective of the paper's Section 3.3.4
// (Eq. 3 clipped objective, Eq. 4 value loss, Eq. 5 their sum with an entropy term): the loss over the
// environments of a mini-batch, then the gradient with respect to every weight, layer by layer backwards
// through the heads, Eq. 8, the k attention layers of Eq. 7 and Eq. 6.
//
// What is in this file: the forward pass of xrl_ppo_grad keeps every layer's input, Z rows and half-scores
// (nothing is recomputed here); the reverse of Eq. 7 runs row-wise kernels (a warp per destination row:
// k_aggregate_bwd_rows, k_scores_bwd_rows) with generic fallbacks (k_aggregate_bwd, k_scores_bwd) for head
// counts that do not divide 32; the two dense products of a layer, dW = h_in^T dz and dh_in = dz W^T, run on
// the tensor cores (mma.sync bf16, fp32 accumulate: k_atb_mma, k_gwt_mma) for bf16 models of hidden 128, 256
// or 512 and on CUDA-core tiles (k_atb, k_gwt) otherwise.  Gradients are fp32; sums over rows are collected
// with floating-point atomics, so the last bits of a gradient depend on the order in which the hardware
// serves them.  Activations saved by the forward pass are read in their storage type.  On the tensor-core
// path the half-score terms (ds a) are added into the bf16 copy of dz that the products read (`dzb`) only:
// the fp32 `dz` buffer is then left without them and must not be read afterwards.
// ReLU'(0) = 0, LeakyReLU'(0) = 0.2; the clipped objective has the slope of whichever term of its min is
// the smaller one.
#include <algorithm>

#include "xrl_internal.cuh"

namespace xrl {

namespace {

__device__ __forceinline__ float lrelu(float x) { return fmaxf(x, 0.2f * x); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Z rows and half-score pairs of a layer, in either layout (pairs behind the rows, or in their own array).
template <typename T> struct ZView {
  const char* z; size_t row_bytes; const float2* pairs; int pair_stride;   // pairs[i * pair_stride + k]
  __device__ __forceinline__ const T* row(int32_t i) const { return reinterpret_cast<const T*>(z + size_t(i) * row_bytes); }
  __device__ __forceinline__ float2 pair(int32_t i, int k) const { return pairs[size_t(i) * pair_stride + k]; }
};

constexpr int kMaxPerLane = 16;          // hidden <= 512

// ---- Eq. 7, reverse: one warp per destination row ---------------------------------------------------
// in : dh_out [N x H] fp32 (gradient of the layer's output), h_out (its output, for the ReLU), Z / pairs
// out: dz [N x H] fp32 += alpha * dpre (scattered to the gathered rows, atomics), ds_src [N x K] += (atomics),
//      ds_dst [N x K] = (own row), db [H] += (atomics, one per CTA and column)
template <typename T>
__global__ void __launch_bounds__(256)
k_aggregate_bwd(const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, ZView<T> zv,
                const T* __restrict__ h_out, const float* __restrict__ dh_out, float* __restrict__ dz,
                float* __restrict__ ds_src, float* __restrict__ ds_dst, float* __restrict__ db, int N, int H,
                int K) {
  extern __shared__ float sm_db[];                 // [H] per-CTA sums of dpre
  for (int c = threadIdx.x; c < H; c += blockDim.x) sm_db[c] = 0.f;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int d = H / K, NF = H / 32;
  for (int32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < N; i += warps) {
    float dp[kMaxPerLane];
#pragma unroll
    for (int f = 0; f < kMaxPerLane; ++f) {
      dp[f] = 0.f;
      if (f < NF) {
        const int c = lane + 32 * f;
        dp[f] = to_float(h_out[size_t(i) * H + c]) > 0.f ? dh_out[size_t(i) * H + c] : 0.f;
        atomicAdd(&sm_db[c], dp[f]);
      }
    }
    const int32_t e0 = rowptr[i], deg = rowptr[i + 1] - e0;
    // softmax statistics per head (every lane keeps all K heads; K is small)
    for (int k0 = 0; k0 < K; ++k0) {
      const float sd = zv.pair(i, k0).y;
      float mx = -INFINITY;
      for (int t = lane; t <= deg; t += 32) {
        const int32_t j = t < deg ? col[e0 + t] : i;
        mx = fmaxf(mx, lrelu(zv.pair(j, k0).x + sd));
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
      float sum = 0.f;
      for (int t = lane; t <= deg; t += 32) {
        const int32_t j = t < deg ? col[e0 + t] : i;
        sum += exp2f(lrelu(zv.pair(j, k0).x + sd) - mx);
      }
      sum = warp_sum(sum);
      const float inv = 1.f / sum;
      // dal_t = sum over the head's features of dpre * z_j; dot = sum_t alpha_t dal_t
      float dot = 0.f;
      for (int t = 0; t <= deg; ++t) {
        const int32_t j = t < deg ? col[e0 + t] : i;
        const T* zj = zv.row(j);
        float part = 0.f;
#pragma unroll
        for (int f = 0; f < kMaxPerLane; ++f)
          if (f < NF) {
            const int c = lane + 32 * f;
            if (c / d == k0) part += dp[f] * to_float(zj[c]);
          }
        const float dal = warp_sum(part);
        const float al = exp2f(lrelu(zv.pair(j, k0).x + sd) - mx) * inv;
        dot += al * dal;
      }
      float dsd = 0.f;
      for (int t = 0; t <= deg; ++t) {
        const int32_t j = t < deg ? col[e0 + t] : i;
        const T* zj = zv.row(j);
        float part = 0.f;
#pragma unroll
        for (int f = 0; f < kMaxPerLane; ++f)
          if (f < NF) {
            const int c = lane + 32 * f;
            if (c / d == k0) part += dp[f] * to_float(zj[c]);
          }
        const float dal = warp_sum(part);
        const float e = zv.pair(j, k0).x + sd;          // (times log2 e: the sign is what matters below)
        const float al = exp2f(lrelu(e) - mx) * inv;
        const float de = al * (dal - dot) * (e > 0.f ? 1.f : 0.2f);
        dsd += de;
        if (lane == 0) atomicAdd(&ds_src[size_t(j) * K + k0], de);
#pragma unroll
        for (int f = 0; f < kMaxPerLane; ++f)
          if (f < NF) {
            const int c = lane + 32 * f;
            if (c / d == k0) atomicAdd(&dz[size_t(j) * H + c], al * dp[f]);
          }
      }
      if (lane == 0) ds_dst[size_t(i) * K + k0] = dsd;
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < H; c += blockDim.x)
    if (sm_db[c] != 0.f) atomicAdd(&db[c], sm_db[c]);
}

// ---- half-scores, reverse: dz += ds_src a_src + ds_dst a_dst; da_src += ds_src z; da_dst += ds_dst z -----
template <typename T>
__global__ void __launch_bounds__(256)
k_scores_bwd(ZView<T> zv, const float* __restrict__ ds_src, const float* __restrict__ ds_dst,
             const float* __restrict__ a_src, const float* __restrict__ a_dst, float* __restrict__ dz,
             float* __restrict__ da_src, float* __restrict__ da_dst, int N, int H, int K) {
  extern __shared__ float sm_da[];                 // [2H]
  for (int c = threadIdx.x; c < 2 * H; c += blockDim.x) sm_da[c] = 0.f;
  __syncthreads();
  const int d = H / K;
  const int rows_per_cta = (N + gridDim.x - 1) / gridDim.x;
  const int r0 = blockIdx.x * rows_per_cta, r1 = min(N, r0 + rows_per_cta);
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    const int k = c / d;
    const float as = a_src[c], ad = a_dst[c];
    float accs = 0.f, accd = 0.f;
    for (int i = r0; i < r1; ++i) {
      const float gs = ds_src[size_t(i) * K + k], gd = ds_dst[size_t(i) * K + k];
      const float z = to_float(zv.row(i)[c]);
      dz[size_t(i) * H + c] += gs * as + gd * ad;
      accs += gs * z;
      accd += gd * z;
    }
    sm_da[c] = accs;
    sm_da[H + c] = accd;
  }
  __syncthreads();
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    atomicAdd(&da_src[c], sm_da[c]);
    atomicAdd(&da_dst[c], sm_da[H + c]);
  }
}

// ---- the same two kernels for the usual shapes: K divides 32 and H = 32 NF, NF in {1, 2, 4, 8, 16} ----------
// A lane owns NF consecutive features, all of one head (32 / K lanes per head): a head's reductions stay inside
// its group of lanes, all heads proceed at once, rows move as 4- to 16-byte pieces, and the scattered sums
// go out as vector atomics.
template <typename T, int NF> struct alignas((sizeof(T) * NF) >= 16 ? 16 : sizeof(T) * NF) Chunk { T v[NF]; };

template <typename T, int NF>
__device__ __forceinline__ void load_chunk(const T* p, float (&f)[NF]) {
  const Chunk<T, NF> c = *reinterpret_cast<const Chunk<T, NF>*>(p);
#pragma unroll
  for (int t = 0; t < NF; ++t) f[t] = to_float(c.v[t]);
}
template <int NF>
__device__ __forceinline__ void store_chunk(float* p, const float (&f)[NF]) {
  Chunk<float, NF> c;
#pragma unroll
  for (int t = 0; t < NF; ++t) c.v[t] = f[t];
  *reinterpret_cast<Chunk<float, NF>*>(p) = c;
}
template <int NF>
__device__ __forceinline__ void atomic_add_chunk(float* p, const float (&v)[NF]) {
  if constexpr (NF % 4 == 0) {
#pragma unroll
    for (int q = 0; q < NF / 4; ++q)
      atomicAdd(reinterpret_cast<float4*>(p) + q, make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]));
  } else if constexpr (NF % 2 == 0) {
#pragma unroll
    for (int q = 0; q < NF / 2; ++q) atomicAdd(reinterpret_cast<float2*>(p) + q, make_float2(v[2 * q], v[2 * q + 1]));
  } else {
#pragma unroll
    for (int q = 0; q < NF; ++q) atomicAdd(p + q, v[q]);
  }
}

template <typename T, int NF>
__global__ void __launch_bounds__(256)
k_aggregate_bwd_rows(const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, ZView<T> zv,
                     const T* __restrict__ h_out, const float* __restrict__ dh_out, float* __restrict__ dz,
                     float* __restrict__ ds_src, float* __restrict__ ds_dst, float* __restrict__ db, int N, int K) {
  constexpr int H = 32 * NF;
  __shared__ float sm_db[H];
  for (int c = threadIdx.x; c < H; c += blockDim.x) sm_db[c] = 0.f;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int lph = 32 / K, k = lane / lph;            // lanes per head, this lane's head
  const bool leader = (lane % lph) == 0;
  float dbr[NF];
#pragma unroll
  for (int f = 0; f < NF; ++f) dbr[f] = 0.f;
  for (int32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < N; i += warps) {
    float dp[NF];
    {
      float g[NF], ho[NF];
      load_chunk<float, NF>(dh_out + size_t(i) * H + lane * NF, g);
      load_chunk<T, NF>(h_out + size_t(i) * H + lane * NF, ho);
#pragma unroll
      for (int f = 0; f < NF; ++f) { dp[f] = ho[f] > 0.f ? g[f] : 0.f; dbr[f] += dp[f]; }
    }
    bool live = false;
#pragma unroll
    for (int f = 0; f < NF; ++f) live = live || dp[f] != 0.f;
    if (!__any_sync(0xFFFFFFFFu, live)) continue;     // a row whose units are all off: nothing flows (ds is zeroed)
    const int32_t e0 = rowptr[i], deg = rowptr[i + 1] - e0;
    const float sd = zv.pair(i, k).y;
    // One sweep over the row's neighbours and the row itself (entry `deg`) takes, per head, the score e_t, the
    // product dal_t = dpre . z_t, and with a running maximum the sums  sum_t 2^(e_t - mx)  and
    // sum_t 2^(e_t - mx) dal_t; the first kCache entries keep (e_t, dal_t) in registers for the second sweep,
    // which turns them into d e_t and the scattered sums (later entries are read and multiplied again).
    constexpr int kCache = 4;
    float ce[kCache], cd[kCache];
    float mx = -INFINITY, sum = 0.f, dotu = 0.f;
    auto product = [&](const Chunk<T, NF>& zc, float& dal) {
      float part = 0.f;
#pragma unroll
      for (int f = 0; f < NF; ++f) part = fmaf(dp[f], to_float(zc.v[f]), part);
      for (int o = lph >> 1; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
      dal = part;
    };
    auto score_and_product = [&](int32_t j, float& eraw, float& dal) {
      const Chunk<T, NF> zc = *reinterpret_cast<const Chunk<T, NF>*>(zv.row(j) + lane * NF);
      eraw = zv.pair(j, k).x + sd;
      product(zc, dal);
    };
    auto accumulate = [&](float eraw, float dal) {
      const float e = lrelu(eraw);
      if (e > mx) {
        const float sc = exp2f(mx - e);
        sum = fmaf(sum, sc, 1.f); dotu = fmaf(dotu, sc, dal); mx = e;
      } else {
        const float w = exp2f(e - mx);
        sum += w; dotu = fmaf(w, dal, dotu);
      }
    };
    const int32_t c0 = lane < deg ? col[e0 + lane] : i;      // the first 32 entries (the row itself after the last)
    {
      // the first kCache rows are fetched together (entries past the last one repeat it: always a valid row)
      Chunk<T, NF> zc[kCache];
#pragma unroll
      for (int t = 0; t < kCache; ++t) {
        const int32_t j = __shfl_sync(0xFFFFFFFFu, c0, min(t, deg));
        zc[t] = *reinterpret_cast<const Chunk<T, NF>*>(zv.row(j) + lane * NF);
        ce[t] = zv.pair(j, k).x;
      }
#pragma unroll
      for (int t = 0; t < kCache; ++t) {
        ce[t] += sd;
        cd[t] = 0.f;
        if (t <= deg) {
          product(zc[t], cd[t]);
          accumulate(ce[t], cd[t]);
        }
      }
    }
    for (int base = 0; base <= deg; base += 32) {
      const int idx = base + lane;
      const int32_t cj = base == 0 ? c0 : (idx < deg ? col[e0 + idx] : i);
      const int cnt = min(32, deg + 1 - base);
      for (int t = (base == 0 ? kCache : 0); t < cnt; ++t) {
        const int32_t j = __shfl_sync(0xFFFFFFFFu, cj, t);
        float eraw, dal;
        score_and_product(j, eraw, dal);
        accumulate(eraw, dal);
      }
    }
    const float inv = 1.f / sum;
    const float dot = dotu * inv;
    float dsd = 0.f;
    auto scatter = [&](int32_t j, float eraw, float dal) {
      const float al = exp2f(lrelu(eraw) - mx) * inv;
      const float de = al * (dal - dot) * (eraw > 0.f ? 1.f : 0.2f);
      dsd += de;
      if (leader && de != 0.f) atomicAdd(&ds_src[size_t(j) * K + k], de);
      if (live) {
        float v[NF];
#pragma unroll
        for (int f = 0; f < NF; ++f) v[f] = al * dp[f];
        atomic_add_chunk<NF>(dz + size_t(j) * H + lane * NF, v);
      }
    };
#pragma unroll
    for (int t = 0; t < kCache; ++t)
      if (t <= deg) scatter(__shfl_sync(0xFFFFFFFFu, c0, t), ce[t], cd[t]);
    for (int base = 0; base <= deg; base += 32) {
      const int idx = base + lane;
      const int32_t cj = base == 0 ? c0 : (idx < deg ? col[e0 + idx] : i);
      const int cnt = min(32, deg + 1 - base);
      for (int t = (base == 0 ? kCache : 0); t < cnt; ++t) {
        const int32_t j = __shfl_sync(0xFFFFFFFFu, cj, t);
        float eraw, dal;
        score_and_product(j, eraw, dal);
        scatter(j, eraw, dal);
      }
    }
    if (leader) ds_dst[size_t(i) * K + k] = dsd;
  }
#pragma unroll
  for (int f = 0; f < NF; ++f)
    if (dbr[f] != 0.f) atomicAdd(&sm_db[lane * NF + f], dbr[f]);
  __syncthreads();
  for (int c = threadIdx.x; c < H; c += blockDim.x)
    if (sm_db[c] != 0.f) atomicAdd(&db[c], sm_db[c]);
}

// dz += ds_src a_src + ds_dst a_dst per row and head, da_src / da_dst += ds z.  With `dzb` (tensor-core
// products follow) the completed row goes to dzb in bf16 and the fp32 dz is NOT updated.
template <typename T, int NF>
__global__ void __launch_bounds__(256)
k_scores_bwd_rows(ZView<T> zv, const float* __restrict__ ds_src, const float* __restrict__ ds_dst,
                  const float* __restrict__ a_src, const float* __restrict__ a_dst, float* __restrict__ dz,
                  bf16* __restrict__ dzb, float* __restrict__ da_src, float* __restrict__ da_dst, int N, int K) {
  constexpr int H = 32 * NF;
  __shared__ float sm_da[2 * H];
  for (int c = threadIdx.x; c < 2 * H; c += blockDim.x) sm_da[c] = 0.f;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int k = lane / (32 / K);
  float as[NF], ad[NF], accs[NF], accd[NF];
  load_chunk<float, NF>(a_src + lane * NF, as);
  load_chunk<float, NF>(a_dst + lane * NF, ad);
#pragma unroll
  for (int f = 0; f < NF; ++f) { accs[f] = 0.f; accd[f] = 0.f; }
  for (int32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < N; i += warps) {
    const float gs = ds_src[size_t(i) * K + k], gd = ds_dst[size_t(i) * K + k];
    float z[NF], g[NF];
    load_chunk<float, NF>(dz + size_t(i) * H + lane * NF, g);
    if (gs != 0.f || gd != 0.f) {
      load_chunk<T, NF>(zv.row(i) + lane * NF, z);
#pragma unroll
      for (int f = 0; f < NF; ++f) {
        g[f] += gs * as[f] + gd * ad[f];
        accs[f] = fmaf(gs, z[f], accs[f]);
        accd[f] = fmaf(gd, z[f], accd[f]);
      }
      if (dzb == nullptr) store_chunk<NF>(dz + size_t(i) * H + lane * NF, g);
    }
    if (dzb != nullptr) {                             // the tensor-core products read dz in bf16
      Chunk<bf16, NF> c;
#pragma unroll
      for (int f = 0; f < NF; ++f) c.v[f] = __float2bfloat16(g[f]);
      *reinterpret_cast<Chunk<bf16, NF>*>(dzb + size_t(i) * H + lane * NF) = c;
    }
  }
#pragma unroll
  for (int f = 0; f < NF; ++f) {
    atomicAdd(&sm_da[lane * NF + f], accs[f]);
    atomicAdd(&sm_da[H + lane * NF + f], accd[f]);
  }
  __syncthreads();
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    if (sm_da[c] != 0.f) atomicAdd(&da_src[c], sm_da[c]);
    if (sm_da[H + c] != 0.f) atomicAdd(&da_dst[c], sm_da[H + c]);
  }
}

// ---- dW += A^T B over a range of rows: A [rows x Ka] (storage type), B [rows x Nb] fp32 -------------------
// 64 x 64 output tile per CTA, the rows cut into chunks along grid.z, partial products added with atomics.
template <typename TA>
__global__ void __launch_bounds__(256)
k_atb(const TA* __restrict__ A, int lda, const float* __restrict__ Bm, int ldb, float* __restrict__ Cout, int ldc,
      int rows, int Ka, int Nb, int rows_per_chunk, float* __restrict__ colsum_out) {
  __shared__ float As[16][64 + 1];
  __shared__ float Bs[16][64 + 1];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int a0 = blockIdx.x * 64, b0 = blockIdx.y * 64;
  const int r_begin = blockIdx.z * rows_per_chunk, r_end = min(rows, r_begin + rows_per_chunk);
  float acc[4][4] = {};
  // with colsum_out the first row of CTAs also sums B's columns (the bias gradient that goes with the product)
  const bool sums = colsum_out != nullptr && blockIdx.x == 0 && ty == 0;
  float csum[4] = {0.f, 0.f, 0.f, 0.f};
  for (int r0 = r_begin; r0 < r_end; r0 += 16) {
    for (int t = tid; t < 16 * 64; t += 256) {
      const int rr = t >> 6, cc = t & 63;
      const int r = r0 + rr;
      As[rr][cc] = (r < r_end && a0 + cc < Ka) ? to_float(A[size_t(r) * lda + a0 + cc]) : 0.f;
      Bs[rr][cc] = (r < r_end && b0 + cc < Nb) ? Bm[size_t(r) * ldb + b0 + cc] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int rr = 0; rr < 16; ++rr) {
      float a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { a[u] = As[rr][ty * 4 + u]; b[u] = Bs[rr][tx * 4 + u]; }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
      if (sums) {
#pragma unroll
        for (int v = 0; v < 4; ++v) csum[v] += b[v];
      }
    }
    __syncthreads();
  }
  if (sums) {
#pragma unroll
    for (int v = 0; v < 4; ++v)
      if (b0 + tx * 4 + v < Nb && csum[v] != 0.f) atomicAdd(&colsum_out[b0 + tx * 4 + v], csum[v]);
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int ka = a0 + ty * 4 + u, nb = b0 + tx * 4 + v;
      if (ka < Ka && nb < Nb && acc[u][v] != 0.f) atomicAdd(&Cout[size_t(ka) * ldc + nb], acc[u][v]);
    }
}

// ---- out = G W^T: G [rows x Hn] fp32, W [Hk x Hn] (storage type, row-major [in x out]) -> out [rows x Hk] ----
template <typename TW>
__global__ void __launch_bounds__(256)
k_gwt(const float* __restrict__ G, const TW* __restrict__ W, float* __restrict__ out, int rows, int Hk, int Hn) {
  __shared__ float Gs[64][16 + 1];
  __shared__ float Ws[64][16 + 1];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int r0 = blockIdx.x * 64, k0 = blockIdx.y * 64;
  float acc[4][4] = {};
  for (int c0 = 0; c0 < Hn; c0 += 16) {
    for (int t = tid; t < 64 * 16; t += 256) {
      const int rr = t >> 4, cc = t & 15;
      Gs[rr][cc] = (r0 + rr < rows && c0 + cc < Hn) ? G[size_t(r0 + rr) * Hn + c0 + cc] : 0.f;
      Ws[rr][cc] = (k0 + rr < Hk && c0 + cc < Hn) ? to_float(W[size_t(k0 + rr) * Hn + c0 + cc]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int cc = 0; cc < 16; ++cc) {
      float g[4], w[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { g[u] = Gs[ty * 4 + u][cc]; w[u] = Ws[tx * 4 + u][cc]; }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(g[u], w[v], acc[u][v]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int r = r0 + ty * 4 + u, k = k0 + tx * 4 + v;
      if (r < rows && k < Hk) out[size_t(r) * Hk + k] = acc[u][v];
    }
}

// ---- the two products of a layer's reverse pass on the tensor cores (bf16 models, H a multiple of 128) --------
// mma.sync m16n8k16, bf16 operands, fp32 accumulators; a CTA of 8 warps (4 x 2) takes a 128 x 128 tile of the
// result, a warp 32 x 64.  Operand tiles sit in shared memory in 16-byte pieces whose position within a row is
// XOR-ed with the row number, so that the eight rows one ldmatrix reads fall into different banks.
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// out [rows x H] fp32 = G [rows x H] bf16 times W^T, W [H x H] bf16 row-major [in x out]: out[r][k] = sum_n G[r][n] W[k][n]
// A CTA takes tiles_per_cta consecutive tiles of 128 rows (kGwtTiles when that still leaves several waves of
// CTAs, else one); its loop runs over (tile, 64-wide step of n) pairs, so
// that the first pieces of the next tile are already on their way while the last step of the current tile is
// multiplied and its 64 KB of results are stored.
constexpr int kGwtTiles = 4;
__global__ void __launch_bounds__(256, 2)
k_gwt_mma(const bf16* __restrict__ G, const bf16* __restrict__ W, float* __restrict__ out, int rows, int H,
          int tiles_per_cta) {
  __shared__ __align__(128) bf16 As[128 * 64];      // [row r][64 n], 8 pieces of 16 bytes per row
  __shared__ __align__(128) bf16 Bs[128 * 64];      // [row k][64 n]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp >> 1, wn = warp & 1;
  // consecutive CTAs take the column tiles of the same rows, so that the rows' second reading comes from L2
  const int ncol = H / 128;
  const int k0 = int(blockIdx.x % ncol) * 128;
  const int tile0 = int(blockIdx.x / ncol) * tiles_per_cta, ntiles = (rows + 127) / 128;
  const int nk = H / 64, total = min(tiles_per_cta, ntiles - tile0) * nk;
  float acc[2][8][4];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
  const uint32_t as_base = uint32_t(__cvta_generic_to_shared(As)), bs_base = uint32_t(__cvta_generic_to_shared(Bs));
  // the next step's pieces travel from global memory to registers while the current step is multiplied
  uint4 va[4], vb[4];
  auto fetch = [&](int step) {
    const int r0 = (tile0 + step / nk) * 128, n0 = (step % nk) * 64;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + 256 * it, row = idx >> 3, ch = idx & 7;
      va[it] = make_uint4(0, 0, 0, 0);
      if (r0 + row < rows) va[it] = *reinterpret_cast<const uint4*>(G + size_t(r0 + row) * H + n0 + ch * 8);
      vb[it] = *reinterpret_cast<const uint4*>(W + size_t(k0 + row) * H + n0 + ch * 8);
    }
  };
  if (total > 0) fetch(0);
  for (int step = 0; step < total; ++step) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + 256 * it, row = idx >> 3, ch = idx & 7;
      const int phys = (row * 8 + (ch ^ (row & 7))) * 8;
      *reinterpret_cast<uint4*>(As + phys) = va[it];
      *reinterpret_cast<uint4*>(Bs + phys) = vb[it];
    }
    __syncthreads();
    if (step + 1 < total) fetch(step + 1);
#pragma unroll
    for (int kk = 0; kk < 64; kk += 16) {
      uint32_t af[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const int row = wm * 32 + mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = (kk >> 3) + (lane >> 4);
        ldsm_x4(af[mt], as_base + uint32_t((row * 8 + (ch ^ (row & 7))) * 16));
      }
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t bf[4];
        const int row = wn * 64 + np * 16 + (lane & 7) + (lane >> 4) * 8;
        const int ch = (kk >> 3) + ((lane >> 3) & 1);
        ldsm_x4(bf, bs_base + uint32_t((row * 8 + (ch ^ (row & 7))) * 16));
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          mma_bf16(acc[mt][2 * np], af[mt], bf[0], bf[1]);
          mma_bf16(acc[mt][2 * np + 1], af[mt], bf[2], bf[3]);
        }
      }
    }
    __syncthreads();
    if (step % nk == nk - 1) {                       // the tile is complete: store it, start the next from zero
      const int r0 = (tile0 + step / nk) * 128;
      const int g = lane >> 2, t = lane & 3;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int r = r0 + wm * 32 + mt * 16 + g, c = k0 + wn * 64 + nt * 8 + 2 * t;
          if (r < rows)
            *reinterpret_cast<float2*>(out + size_t(r) * H + c) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
          if (r + 8 < rows)
            *reinterpret_cast<float2*>(out + size_t(r + 8) * H + c) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
#pragma unroll
          for (int q = 0; q < 4; ++q) acc[mt][nt][q] = 0.f;
        }
    }
  }
}

// dW [H x H] fp32 += A^T B over the rows [chunk z], A = h_in [rows x H] bf16, B = dz [rows x H] bf16
__global__ void __launch_bounds__(256, 2)
k_atb_mma(const bf16* __restrict__ A, const bf16* __restrict__ Bm, float* __restrict__ dW, int rows, int H,
          int rows_per_chunk) {
  __shared__ __align__(128) bf16 As[32 * 128];      // [row r][128 m], 16 pieces of 16 bytes per row
  __shared__ __align__(128) bf16 Bs[32 * 128];      // [row r][128 n]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp >> 1, wn = warp & 1;
  const int m0 = blockIdx.x * 128, n0 = blockIdx.y * 128;
  const int r_begin = blockIdx.z * rows_per_chunk, r_end = min(rows, r_begin + rows_per_chunk);
  float acc[2][8][4];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
  const uint32_t as_base = uint32_t(__cvta_generic_to_shared(As)), bs_base = uint32_t(__cvta_generic_to_shared(Bs));
  uint4 va[2], vb[2];
  auto fetch = [&](int rr) {
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int idx = tid + 256 * it, row = idx >> 4, ch = idx & 15;
      va[it] = make_uint4(0, 0, 0, 0); vb[it] = make_uint4(0, 0, 0, 0);
      if (rr + row < r_end) {
        va[it] = *reinterpret_cast<const uint4*>(A + size_t(rr + row) * H + m0 + ch * 8);
        vb[it] = *reinterpret_cast<const uint4*>(Bm + size_t(rr + row) * H + n0 + ch * 8);
      }
    }
  };
  if (r_begin < r_end) fetch(r_begin);
  for (int rr = r_begin; rr < r_end; rr += 32) {
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const int idx = tid + 256 * it, row = idx >> 4, ch = idx & 15;
      const int phys = (row * 16 + (ch ^ (row & 7))) * 8;
      *reinterpret_cast<uint4*>(As + phys) = va[it];
      *reinterpret_cast<uint4*>(Bs + phys) = vb[it];
    }
    __syncthreads();
    if (rr + 32 < r_end) fetch(rr + 32);
#pragma unroll
    for (int kk = 0; kk < 32; kk += 16) {
      uint32_t af[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        // the stored rows are the products' k index: transposed 8 x 8 loads give the (m, k) fragments
        const int row = kk + (lane & 7) + (lane >> 4) * 8;
        const int ch = ((wm * 32 + mt * 16) >> 3) + ((lane >> 3) & 1);
        ldsm_x4_trans(af[mt], as_base + uint32_t((row * 16 + (ch ^ (row & 7))) * 16));
      }
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t bf[4];
        const int row = kk + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ch = ((wn * 64 + np * 16) >> 3) + (lane >> 4);
        ldsm_x4_trans(bf, bs_base + uint32_t((row * 16 + (ch ^ (row & 7))) * 16));
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          mma_bf16(acc[mt][2 * np], af[mt], bf[0], bf[1]);
          mma_bf16(acc[mt][2 * np + 1], af[mt], bf[2], bf[3]);
        }
      }
    }
    __syncthreads();
  }
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int m = m0 + wm * 32 + mt * 16 + g, n = n0 + wn * 64 + nt * 8 + 2 * t;
      float* o = dW + size_t(m) * H + n;
      if (acc[mt][nt][0] != 0.f) atomicAdd(o, acc[mt][nt][0]);
      if (acc[mt][nt][1] != 0.f) atomicAdd(o + 1, acc[mt][nt][1]);
      if (acc[mt][nt][2] != 0.f) atomicAdd(o + size_t(8) * H, acc[mt][nt][2]);
      if (acc[mt][nt][3] != 0.f) atomicAdd(o + size_t(8) * H + 1, acc[mt][nt][3]);
    }
}

// the sixteen dense entries of Eq. 6's input, one thread per node: [sum of the edge attributes | own shape]
template <typename T>
__global__ void __launch_bounds__(256)
k_embed_inputs(const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col, const T* __restrict__ shape,
               const T* __restrict__ eattr, float* __restrict__ xs, int N) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  float x[2 * kS];
#pragma unroll
  for (int s = 0; s < kS; ++s) x[s] = 0.f;
  for (int32_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
    float v[kS];
    load_chunk<T, kS>(eattr ? eattr + size_t(e) * kS : shape + size_t(col[e]) * kS, v);
#pragma unroll
    for (int s = 0; s < kS; ++s) x[s] += v[s];
  }
  load_chunk<T, kS>(shape + size_t(i) * kS, reinterpret_cast<float(&)[kS]>(x[kS]));
  store_chunk<2 * kS>(xs + size_t(i) * 2 * kS, x);
}

// ---- Eq. 6, reverse: dW0 += x^T dpre, db0 += dpre, x_i = [edge sum | one-hot op | own shape] -------------
// A CTA takes a range of rows, R at a time: the tile's masked gradients dpre [R x H], its dense inputs
// [R x 16] (computed beforehand by k_embed_inputs) and its operator ids come into shared memory with wide
// coalesced loads, eight requested per thread before the first is used; then a thread owns one column and
// every P-th row of the tile (P threads share a column): the sixteen dense products accumulate in its
// registers, the one-hot block in the P-th of P shared-memory copies [T x H] of that part of dW0 (a plain add
// per row and column: nobody else touches that copy's column; shared-memory atomics cost far more here than
// the adds themselves).  Registers and the copies go to global memory once per CTA.
constexpr int kEmbedBwdThreads = 512;
template <typename T>
__global__ void __launch_bounds__(kEmbedBwdThreads)
k_embed_bwd(const float* __restrict__ xs, const int32_t* __restrict__ op, const T* __restrict__ h0,
            const float* __restrict__ dh0, float* __restrict__ dW0, float* __restrict__ db0, int N, int H, int Tn,
            int R, int P) {
  extern __shared__ float sm_embed[];
  float* oh = sm_embed;                            // [P][Tn x H]
  float* dpt = oh + size_t(P) * Tn * H;            // [R x H]
  float* xt = dpt + size_t(R) * H;                 // [R x 16]
  int32_t* opt = reinterpret_cast<int32_t*>(xt + size_t(R) * 2 * kS);   // [R]
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int t = tid; t < P * Tn * H; t += nt) oh[t] = 0.f;
  const int part = tid / H, c = tid - part * H;    // threads beyond P x H only help with the loads
  float* my_oh = oh + size_t(min(part, P - 1)) * Tn * H;
  const int rows_per_cta = (N + gridDim.x - 1) / gridDim.x;
  const int r0 = blockIdx.x * rows_per_cta, r1 = min(N, r0 + rows_per_cta);
  const int qpr = H >> 2;                          // 16-byte pieces per row
  const int step_r = nt / qpr, step_q = nt - step_r * qpr;   // what a stride of nt pieces does to (row, piece)
  float acc[2 * kS], dbr = 0.f;
#pragma unroll
  for (int s = 0; s < 2 * kS; ++s) acc[s] = 0.f;
  for (int t0 = r0; t0 < r1; t0 += R) {
    const int rows = min(R, r1 - t0);
    __syncthreads();                               // the previous tile has been consumed (and oh is zeroed)
    constexpr int kBatch = 8;
    int r = tid / qpr, q = tid - r * qpr;
    while (r < rows) {
      float4 g[kBatch];
      Chunk<T, 4> hc[kBatch];
      int rr[kBatch], qq[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        rr[u] = r; qq[u] = q;
        if (r < rows) {
          g[u] = *reinterpret_cast<const float4*>(dh0 + size_t(t0 + r) * H + 4 * q);
          hc[u] = *reinterpret_cast<const Chunk<T, 4>*>(h0 + size_t(t0 + r) * H + 4 * q);
        }
        r += step_r; q += step_q;
        if (q >= qpr) { q -= qpr; ++r; }
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u)
        if (rr[u] < rows)
          *reinterpret_cast<float4*>(dpt + size_t(rr[u]) * H + 4 * qq[u]) =
              make_float4(to_float(hc[u].v[0]) > 0.f ? g[u].x : 0.f, to_float(hc[u].v[1]) > 0.f ? g[u].y : 0.f,
                          to_float(hc[u].v[2]) > 0.f ? g[u].z : 0.f, to_float(hc[u].v[3]) > 0.f ? g[u].w : 0.f);
    }
    for (int idx = tid; idx < rows * 4; idx += nt)
      reinterpret_cast<float4*>(xt)[idx] = reinterpret_cast<const float4*>(xs + size_t(t0) * 2 * kS)[idx];
    for (int idx = tid; idx < rows; idx += nt) opt[idx] = min(max(op[t0 + idx], 0), Tn - 1);   // (pack reports bad ids)
    __syncthreads();
    if (part < P) {
      for (int rw = part; rw < rows; rw += P) {
        const float dp = dpt[size_t(rw) * H + c];
        if (dp == 0.f) continue;
        const float4* xr = reinterpret_cast<const float4*>(xt + size_t(rw) * 2 * kS);
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const float4 x = xr[v];
          acc[4 * v] = fmaf(x.x, dp, acc[4 * v]);
          acc[4 * v + 1] = fmaf(x.y, dp, acc[4 * v + 1]);
          acc[4 * v + 2] = fmaf(x.z, dp, acc[4 * v + 2]);
          acc[4 * v + 3] = fmaf(x.w, dp, acc[4 * v + 3]);
        }
        my_oh[size_t(opt[rw]) * H + c] += dp;
        dbr += dp;
      }
    }
  }
  if (part < P) {
#pragma unroll
    for (int s = 0; s < kS; ++s) {
      if (acc[s] != 0.f) atomicAdd(&dW0[size_t(s) * H + c], acc[s]);
      if (acc[kS + s] != 0.f) atomicAdd(&dW0[size_t(kS + Tn + s) * H + c], acc[kS + s]);
    }
    if (dbr != 0.f) atomicAdd(&db0[c], dbr);
  }
  __syncthreads();
  for (int t = tid; t < Tn * H; t += nt) {
    float v = 0.f;
    for (int pp = 0; pp < P; ++pp) v += oh[size_t(pp) * Tn * H + t];
    if (v != 0.f) atomicAdd(&dW0[size_t(kS) * H + t], v);
  }
}

// ---- the heads' MLPs: Linear(in, hid), ReLU, [Linear(hid, hid2), ReLU,] Linear(last, 1) ---------------------
// One CTA per input row.  The forward keeps the hidden activations; the reverse pass turns d(out) into the
// gradients of the hidden pre-activations (d1, d2) and of the input (dx).  The weights' gradients are
// products of those per-row buffers (X^T D1, Y1^T D2, ...), taken afterwards by k_atb (which also sums the columns of D for the biases).
struct MlpW { const float *W1, *b1, *Wh, *bh, *w2, *b2; int hid, hid2; };

__device__ float block_sum_f(float v, float* scratch) {       // blockDim a power of two
  scratch[threadIdx.x] = v;
  __syncthreads();
  for (int s = blockDim.x >> 1; s > 0; s >>= 1) {
    if (int(threadIdx.x) < s) scratch[threadIdx.x] += scratch[threadIdx.x + s];
    __syncthreads();
  }
  const float r = scratch[0];
  __syncthreads();
  return r;
}

// x [in], y1 [hid], y2 [hid2] in shared memory; returns the head's output to every thread
__device__ float mlp_fwd(const float* x, int in, const MlpW& m, float* y1, float* y2, float* scratch) {
  for (int c = threadIdx.x; c < m.hid; c += blockDim.x) {
    float acc = m.b1[c];
#pragma unroll 16
    for (int k = 0; k < in; ++k) acc = fmaf(x[k], m.W1[size_t(k) * m.hid + c], acc);
    y1[c] = fmaxf(acc, 0.f);
  }
  __syncthreads();
  float contrib = 0.f;
  if (m.hid2 <= 0) {
    for (int c = threadIdx.x; c < m.hid; c += blockDim.x) contrib += y1[c] * m.w2[c];
  } else {
    for (int c = threadIdx.x; c < m.hid2; c += blockDim.x) {
      float acc = m.bh[c];
#pragma unroll 16
      for (int k = 0; k < m.hid; ++k) acc = fmaf(y1[k], m.Wh[size_t(k) * m.hid2 + c], acc);
      y2[c] = fmaxf(acc, 0.f);
      contrib += y2[c] * m.w2[c];
    }
  }
  return block_sum_f(contrib, scratch) + m.b2[0];
}

// y1, y2, d1, d2, dx in shared memory (dx [in], may be null)
__device__ void mlp_bwd(int in, const MlpW& m, const float* y1, const float* y2, float dout, float* d1, float* d2,
                        float* dx) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (m.hid2 <= 0) {
    for (int c = threadIdx.x; c < m.hid; c += blockDim.x) d1[c] = y1[c] > 0.f ? m.w2[c] * dout : 0.f;
  } else {
    for (int c = threadIdx.x; c < m.hid2; c += blockDim.x) d2[c] = y2[c] > 0.f ? m.w2[c] * dout : 0.f;
    __syncthreads();
    for (int k = warp; k < m.hid; k += nw) {
      float part = 0.f;
      for (int c = lane; c < m.hid2; c += 32) part = fmaf(m.Wh[size_t(k) * m.hid2 + c], d2[c], part);
      part = warp_sum(part);
      if (lane == 0) d1[k] = y1[k] > 0.f ? part : 0.f;
    }
  }
  __syncthreads();
  if (dx != nullptr) {
    for (int k = warp; k < in; k += nw) {
      float part = 0.f;
      for (int c = lane; c < m.hid; c += 32) part = fmaf(m.W1[size_t(k) * m.hid + c], d1[c], part);
      part = warp_sum(part);
      if (lane == 0) dx[k] = part;
    }
  }
  __syncthreads();
}

// per-graph sums of the last layer's node features into the first H entries of row g of U [B x (H + Dg)] (zeroed
// beforehand): a CTA takes 64 consecutive rows, a thread a column; a run of rows of one graph is summed in a
// register and added to U once (atomics: a graph's rows span several CTAs)
template <typename T>
__global__ void __launch_bounds__(256)
k_graph_sum(const T* __restrict__ h, const int32_t* __restrict__ seg_id, float* __restrict__ U, int N, int H, int HU,
            int rows_per_cta) {
  const int r0 = blockIdx.x * rows_per_cta, r1 = min(N, r0 + rows_per_cta);
  if (r0 >= r1) return;
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    float s = 0.f;
    int32_t g = seg_id[r0];
    for (int i = r0; i < r1; ++i) {
      const int32_t gi = seg_id[i];
      if (gi != g) {
        atomicAdd(&U[size_t(g) * HU + c], s);
        s = 0.f;
        g = gi;
      }
      s += to_float(h[size_t(i) * H + c]);
    }
    atomicAdd(&U[size_t(g) * HU + c], s);
  }
}

// ---- per graph, forward: Eq. 8 and the policy head ---------------------------------------------------------
__global__ void __launch_bounds__(256)
k_graph_fwd(float* __restrict__ U, const float* __restrict__ g0, const float* __restrict__ Wg,
            const float* __restrict__ bg, MlpW pm, float* __restrict__ emb, float* __restrict__ py1,
            float* __restrict__ py2, float* __restrict__ logit, int H, int Dg) {
  extern __shared__ float sm[];
  float* scratch = sm;                              // [blockDim]
  float* uu = scratch + blockDim.x;                 // [H + Dg]
  float* x = uu + H + Dg;                           // [H]
  float* y1 = x + H;                                // [hid]
  float* y2 = y1 + pm.hid;                          // [hid2]
  const int g = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  for (int k = tid; k < H; k += nt) uu[k] = U[size_t(g) * (H + Dg) + k];
  for (int k = tid; k < Dg; k += nt) {              // the graph's global attributes complete its row of U
    const float v = g0 ? g0[size_t(g) * Dg + k] : 0.f;
    uu[H + k] = v;
    U[size_t(g) * (H + Dg) + H + k] = v;
  }
  __syncthreads();
  for (int c = tid; c < H; c += nt) {
    float acc = bg[c];
#pragma unroll 16
    for (int k = 0; k < H + Dg; ++k) acc = fmaf(uu[k], Wg[size_t(k) * H + c], acc);
    x[c] = fmaxf(acc, 0.f);
    emb[size_t(g) * H + c] = x[c];
  }
  __syncthreads();
  const float out = mlp_fwd(x, H, pm, y1, y2, scratch);
  for (int c = tid; c < pm.hid; c += nt) py1[size_t(g) * pm.hid + c] = y1[c];
  for (int c = tid; c < pm.hid2; c += nt) py2[size_t(g) * pm.hid2 + c] = y2[c];
  if (tid == 0) logit[g] = out;
}

// ---- per environment: Eq. 3-5, d J / d logit of its graphs, value head forward and reverse -----------------
// loss[4] += {J, L_clip, L_vf, L_ent} (atomics); dlogit [B]; demb [B x H] = the value head's share (plain
// stores: a graph belongs to one environment); the value head's per-row buffers vu [2H], vy1, vy2, vd1, vd2,
// vdout; logp_out [num_envs].
struct EnvBufs { float *vu, *vy1, *vy2, *vd1, *vd2, *vdout; };

__global__ void __launch_bounds__(256)
k_ppo_env(const float* __restrict__ emb, const float* __restrict__ logit, const int32_t* __restrict__ env_off,
          const uint8_t* __restrict__ mask, const int32_t* __restrict__ action, const float* __restrict__ logp_old,
          const float* __restrict__ adv, const float* __restrict__ ret, float eps, float c1, float c2, MlpW vm,
          EnvBufs eb, int H, int A, int num_envs, float* __restrict__ loss, float* __restrict__ dlogit,
          float* __restrict__ demb, float* __restrict__ logp_out, int32_t* status) {
  extern __shared__ float sm[];
  float* scratch = sm;                              // [blockDim]
  float* u = scratch + blockDim.x;                  // [2H]
  float* du = u + 2 * H;                            // [2H]
  float* y1 = du + 2 * H;                           // [hid]
  float* y2 = y1 + vm.hid;                          // [hid2]
  float* d1 = y2 + vm.hid2;                         // [hid]
  float* d2 = d1 + vm.hid;                          // [hid2]
  const int e = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const int32_t cur = env_off[e];
  const int32_t C = env_off[e + 1] - cur - 1;
  const uint8_t* mk = mask + size_t(e) * A;
  const float inv_ne = 1.f / float(num_envs);
  auto valid = [&](int a) { return a == A || (a < C && mk[a]); };
  auto lg = [&](int a) { return logit[a == A ? cur : cur + 1 + a]; };
  // masked softmax statistics
  float mx = -INFINITY;
  for (int a = tid; a <= A; a += nt)
    if (valid(a)) mx = fmaxf(mx, lg(a));
  scratch[tid] = mx;
  __syncthreads();
  for (int s = nt >> 1; s > 0; s >>= 1) {
    if (tid < s) scratch[tid] = fmaxf(scratch[tid], scratch[tid + s]);
    __syncthreads();
  }
  mx = scratch[0];
  __syncthreads();
  float se = 0.f;
  for (int a = tid; a <= A; a += nt)
    if (valid(a)) se += expf(lg(a) - mx);
  const float sum = block_sum_f(se, scratch);
  const float lsum = logf(sum);
  float pl = 0.f;                                   // sum_a p_a log p_a
  for (int a = tid; a <= A; a += nt)
    if (valid(a)) { const float lp = lg(a) - mx - lsum; pl += expf(lp) * lp; }
  const float plogp = block_sum_f(pl, scratch);
  const int act = action[e];
  if (act < 0 || act > A || !valid(act)) {          // the same for every thread of the CTA
    if (tid == 0) raise(status, XRL_ERR_INVALID_ARG);
    return;
  }
  const float logp = lg(act) - mx - lsum;
  const float ratio = expf(logp - logp_old[e]);
  const float clipped = fminf(fmaxf(ratio, 1.f - eps), 1.f + eps);
  const float t1 = ratio * adv[e], t2 = clipped * adv[e];
  const float dlogp = (t1 <= t2) ? -adv[e] * ratio * inv_ne : 0.f;
  for (int a = tid; a <= A; a += nt) {
    if (a < A && a >= C) continue;                  // no graph behind a padded slot
    const int32_t g = a == A ? cur : cur + 1 + a;
    float dl = 0.f;
    if (valid(a)) {
      const float lp = lg(a) - mx - lsum, p = expf(lp);
      dl = dlogp * ((a == act ? 1.f : 0.f) - p) + c2 * inv_ne * p * (lp - plogp);
    }
    dlogit[g] = dl;
  }
  // value head over [ current graph | mean of the valid candidates ]
  for (int c = tid; c < H; c += nt) u[c] = emb[size_t(cur) * H + c];
  float cnt = 0.f;
  for (int a = tid; a < C; a += nt) cnt += mk[a] ? 1.f : 0.f;
  const float nv = block_sum_f(cnt, scratch);
  for (int c = tid; c < H; c += nt) {
    float s = 0.f;
    for (int a = 0; a < C; ++a)
      if (mk[a]) s += emb[size_t(cur + 1 + a) * H + c];
    u[H + c] = nv > 0.f ? s / nv : 0.f;
  }
  __syncthreads();
  const float v = mlp_fwd(u, 2 * H, vm, y1, y2, scratch);
  const float dv = c1 * 2.f * (v - ret[e]) * inv_ne;
  mlp_bwd(2 * H, vm, y1, y2, dv, d1, d2, du);
  for (int c = tid; c < 2 * H; c += nt) eb.vu[size_t(e) * 2 * H + c] = u[c];
  for (int c = tid; c < vm.hid; c += nt) {
    eb.vy1[size_t(e) * vm.hid + c] = y1[c];
    eb.vd1[size_t(e) * vm.hid + c] = d1[c];
  }
  for (int c = tid; c < vm.hid2; c += nt) {
    eb.vy2[size_t(e) * vm.hid2 + c] = y2[c];
    eb.vd2[size_t(e) * vm.hid2 + c] = d2[c];
  }
  for (int c = tid; c < H; c += nt) {
    demb[size_t(cur) * H + c] = du[c];
    const float share = nv > 0.f ? du[H + c] / nv : 0.f;
    for (int a = 0; a < C; ++a) demb[size_t(cur + 1 + a) * H + c] = mk[a] ? share : 0.f;
  }
  if (tid == 0) {
    eb.vdout[e] = dv;
    const float lc = -(t1 <= t2 ? t1 : t2) * inv_ne, lv = (v - ret[e]) * (v - ret[e]) * inv_ne, le = plogp * inv_ne;
    atomicAdd(&loss[1], lc); atomicAdd(&loss[2], lv); atomicAdd(&loss[3], le);
    atomicAdd(&loss[0], lc + c1 * lv + c2 * le);
    if (logp_out) logp_out[e] = logp;
  }
}

// ---- per graph, reverse: policy head, then Eq. 8 -------------------------------------------------------------
// in : demb (the value head's share), dlogit, emb, py1, py2   out: pd1, pd2, dpre [B x H] (gradient of Eq. 8's
// pre-activation), dr [B x H] (gradient of the graph's readout sum)
__global__ void __launch_bounds__(256)
k_graph_bwd(const float* __restrict__ emb, const float* __restrict__ dlogit, MlpW pm,
            const float* __restrict__ py1, const float* __restrict__ py2, const float* __restrict__ demb,
            const float* __restrict__ Wg, float* __restrict__ pd1, float* __restrict__ pd2,
            float* __restrict__ dpre, float* __restrict__ dr, int H) {
  extern __shared__ float sm[];
  float* dx = sm;                                   // [H]
  float* y1 = dx + H;
  float* y2 = y1 + pm.hid;
  float* d1 = y2 + pm.hid2;
  float* d2 = d1 + pm.hid;
  const int g = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  for (int c = tid; c < pm.hid; c += nt) y1[c] = py1[size_t(g) * pm.hid + c];
  for (int c = tid; c < pm.hid2; c += nt) y2[c] = py2[size_t(g) * pm.hid2 + c];
  __syncthreads();
  mlp_bwd(H, pm, y1, y2, dlogit[g], d1, d2, dx);
  for (int c = tid; c < pm.hid; c += nt) pd1[size_t(g) * pm.hid + c] = d1[c];
  for (int c = tid; c < pm.hid2; c += nt) pd2[size_t(g) * pm.hid2 + c] = d2[c];
  for (int c = tid; c < H; c += nt) {
    const float de = demb[size_t(g) * H + c] + dx[c];
    const float dp = emb[size_t(g) * H + c] > 0.f ? de : 0.f;
    dx[c] = dp;
    dpre[size_t(g) * H + c] = dp;
  }
  __syncthreads();
  for (int k = warp; k < H; k += nw) {
    float part = 0.f;
    for (int c = lane; c < H; c += 32) part = fmaf(Wg[size_t(k) * H + c], dx[c], part);
    part = warp_sum(part);
    if (lane == 0) dr[size_t(g) * H + k] = part;
  }
}

// the readout is a plain sum: every node receives its graph's gradient (four columns per thread; H % 4 == 0)
__global__ void k_readout_bwd(const float* __restrict__ dr, const int32_t* __restrict__ seg_id,
                              float* __restrict__ dh, int64_t n_quads, int H) {
  const int q = H >> 2;
  for (int64_t t = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; t < n_quads; t += int64_t(gridDim.x) * blockDim.x) {
    const int64_t i = t / q;
    const int c = int(t - i * q);
    reinterpret_cast<float4*>(dh)[t] = reinterpret_cast<const float4*>(dr + size_t(seg_id[i]) * H)[c];
  }
}

// rows per chunk such that the chunks of `rows` fit the grid's y / z extent
int chunk_rows(int64_t rows, int at_least) {
  const int64_t need = ((rows + 16383) / 16384 + 15) & ~int64_t(15);
  return int(std::max<int64_t>(at_least, need));
}

void atb_f32(const float* A, int lda, const float* Bm, int ldb, float* Cout, int ldc, int rows, int Ka, int Nb,
             cudaStream_t st, float* colsum_out = nullptr) {
  if (rows <= 0 || Ka <= 0 || Nb <= 0) return;
  const int chunk = chunk_rows(rows, 1024);
  dim3 g(unsigned((Ka + 63) / 64), unsigned((Nb + 63) / 64), unsigned((rows + chunk - 1) / chunk));
  k_atb<float><<<g, 256, 0, st>>>(A, lda, Bm, ldb, Cout, ldc, rows, Ka, Nb, chunk, colsum_out);
}
// weights' gradients of one head from its per-row buffers; returns the launches
int mlp_weight_grads(const float* X, int in, int rows, int hid, int hid2, const float* Y1, const float* Y2,
                     const float* D1, const float* D2, const float* dout, float* gW1, float* gb1, float* gWh,
                     float* gbh, float* gw2, float* gb2, cudaStream_t st) {
  int n = 0;
  atb_f32(X, in, D1, hid, gW1, hid, rows, in, hid, st, gb1); ++n;
  if (hid2 > 0) {
    atb_f32(Y1, hid, D2, hid2, gWh, hid2, rows, hid, hid2, st, gbh); ++n;
    atb_f32(Y2, hid2, dout, 1, gw2, 1, rows, hid2, 1, st, gb2); ++n;
  } else {
    atb_f32(Y1, hid, dout, 1, gw2, 1, rows, hid, 1, st, gb2); ++n;
  }
  return n;
}

// Generalised advantage estimates: one thread per trajectory, backwards over its T steps (a first-order
// recurrence; trajectories are laid out step-major, [T x M], so that the threads of a warp read neighbours)
__global__ void k_gae(const float* __restrict__ reward, const float* __restrict__ values,
                      const uint8_t* __restrict__ done, float gamma, float lambda, int T, int M,
                      float* __restrict__ adv, float* __restrict__ ret) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= M) return;
  float run = 0.f, vnext = values[size_t(T) * M + j];
  for (int t = T - 1; t >= 0; --t) {
    const float nd = done[size_t(t) * M + j] ? 0.f : 1.f;
    const float v = values[size_t(t) * M + j];
    const float delta = reward[size_t(t) * M + j] + gamma * vnext * nd - v;
    run = delta + gamma * lambda * nd * run;
    adv[size_t(t) * M + j] = run;
    ret[size_t(t) * M + j] = run + v;
    vnext = v;
  }
}

}  // namespace

// ---- launchers ------------------------------------------------------------------------------------------
// ---- weights of a rank's means in the data-parallel exchange --------------------------------------------
// buf = [grad * n | loss[0..3] * n | n] before the caller's sum all-reduce; grad, loss = buf / buf[last] after it.
namespace {
template <typename F>
__global__ void k_grad_weigh(const F* __restrict__ grad, int64_t count, const F* __restrict__ loss, F n,
                             F* __restrict__ buf) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < count) buf[i] = grad[i] * n;
  else if (i < count + 4) buf[i] = loss[i - count] * n;
  else if (i == count + 4) buf[i] = n;
}
template <typename F>
__global__ void k_grad_unweigh(const F* __restrict__ buf, int64_t count, F* __restrict__ grad, F* __restrict__ loss) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const F total = buf[count + 4];
  if (i < count) grad[i] = buf[i] / total;
  else if (i < count + 4) loss[i - count] = buf[i] / total;
}
}  // namespace

int launch_grad_weigh(int elem_bytes, const void* grad, int64_t count, const void* loss, int64_t n, void* buf,
                      cudaStream_t st) {
  const unsigned blocks = unsigned((count + 5 + 255) / 256);
  if (elem_bytes == 8)
    k_grad_weigh<double><<<blocks, 256, 0, st>>>(static_cast<const double*>(grad), count,
                                                 static_cast<const double*>(loss), double(n), static_cast<double*>(buf));
  else
    k_grad_weigh<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(grad), count,
                                                static_cast<const float*>(loss), float(n), static_cast<float*>(buf));
  return 1;
}
int launch_grad_unweigh(int elem_bytes, const void* buf, int64_t count, void* grad, void* loss, cudaStream_t st) {
  const unsigned blocks = unsigned((count + 4 + 255) / 256);
  if (elem_bytes == 8)
    k_grad_unweigh<double><<<blocks, 256, 0, st>>>(static_cast<const double*>(buf), count, static_cast<double*>(grad),
                                                   static_cast<double*>(loss));
  else
    k_grad_unweigh<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(buf), count, static_cast<float*>(grad),
                                                  static_cast<float*>(loss));
  return 1;
}

int launch_gae(const float* reward, const float* values, const uint8_t* done, float gamma, float lambda, int32_t T,
               int32_t M, float* adv, float* ret, cudaStream_t st) {
  if (T <= 0 || M <= 0) return 0;
  k_gae<<<unsigned((M + 127) / 128), 128, 0, st>>>(reward, values, done, gamma, lambda, T, M, adv, ret);
  return 1;
}

// every piece of the heads' workspace starts on a 16-byte boundary (some are read as float4)
static size_t up4(size_t n) { return (n + 3) & ~size_t(3); }
size_t ppo_heads_workspace_floats(const Dims& d, int64_t B, int64_t num_envs) {
  const size_t H = d.H, Hm = d.Hm, Hm2 = d.Hm2, b = size_t(B), e = size_t(num_envs);
  return up4(b * (H + d.Dg)) + 4 * up4(b * H) + 2 * up4(b) + 2 * up4(b * Hm) + 2 * up4(b * Hm2) +
         up4(e * 2 * H) + 2 * up4(e * Hm) + 2 * up4(e * Hm2) + up4(e);
}

// Forward from the saved last-layer features to the logits, Eq. 3-5, and the reverse pass down to the gradient
// of the last layer's node features (dh [N x H]).  ws: ppo_heads_workspace_floats floats.
int launch_ppo_heads(const Dims& d, const DevWeights& w, float* grad_base, const float* w_base, const void* hL,
                     const int32_t* node_off, const int32_t* seg_id, const float* g0, const int32_t* env_off,
                     const uint8_t* mask, const int32_t* action, const float* logp_old, const float* adv,
                     const float* ret, float eps, float c1, float c2, int32_t B, int32_t num_envs, int64_t N,
                     float* ws, float* loss, float* dh, float* logp_out, int32_t* status, cudaStream_t st) {
  if (B <= 0 || num_envs <= 0) return 0;
  const size_t H = d.H, Hm = d.Hm, Hm2 = d.Hm2, HU = H + d.Dg;
  float* p = ws;
  auto take = [&](size_t n) { float* q = p; p += up4(n); return q; };
  float* U = take(size_t(B) * HU);
  float* emb = take(size_t(B) * H);
  float* demb = take(size_t(B) * H);
  float* dpre = take(size_t(B) * H);
  float* dr = take(size_t(B) * H);
  float* logit = take(B);
  float* dlogit = take(B);
  float* py1 = take(size_t(B) * Hm);
  float* pd1 = take(size_t(B) * Hm);
  float* py2 = take(size_t(B) * Hm2);
  float* pd2 = take(size_t(B) * Hm2);
  EnvBufs eb;
  eb.vu = take(size_t(num_envs) * 2 * H);
  eb.vy1 = take(size_t(num_envs) * Hm); eb.vd1 = take(size_t(num_envs) * Hm);
  eb.vy2 = take(size_t(num_envs) * Hm2); eb.vd2 = take(size_t(num_envs) * Hm2);
  eb.vdout = take(num_envs);
  auto gp = [&](const float* q) { return grad_base + (q - w_base); };     // same place in the gradient blob
  const MlpW vm{w.vW1, w.vb1, w.vWh, w.vbh, w.vw2, w.vb2, d.Hm, d.Hm2};
  const MlpW pm{w.pW1, w.pb1, w.pWh, w.pbh, w.pw2, w.pb2, d.Hm, d.Hm2};
  int n = 0;
  // one clearing of everything taken above: the per-graph sums are accumulated with atomics, and a bad action
  // leaves its environment's rows unwritten
  cudaMemsetAsync(ws, 0, sizeof(float) * size_t(p - ws), st);
  if (N > 0) {
    const int rows_per_cta = 64;
    const unsigned grid = unsigned((N + rows_per_cta - 1) / rows_per_cta);
    if (d.dtype == XRL_BF16)
      k_graph_sum<bf16><<<grid, 256, 0, st>>>(static_cast<const bf16*>(hL), seg_id, U, int(N), d.H, int(HU), rows_per_cta);
    else
      k_graph_sum<float><<<grid, 256, 0, st>>>(static_cast<const float*>(hL), seg_id, U, int(N), d.H, int(HU),
                                               rows_per_cta);
    ++n;
  }
  k_graph_fwd<<<B, 256, sizeof(float) * (256 + HU + H + Hm + Hm2), st>>>(U, g0, w.Wg, w.bg, pm, emb, py1, py2, logit,
                                                                          d.H, d.Dg);
  ++n;
  k_ppo_env<<<num_envs, 256, sizeof(float) * (256 + 4 * H + 2 * Hm + 2 * Hm2), st>>>(
      emb, logit, env_off, mask, action, logp_old, adv, ret, eps, c1, c2, vm, eb, d.H, d.A, num_envs, loss, dlogit,
      demb, logp_out, status);
  ++n;
  k_graph_bwd<<<B, 256, sizeof(float) * (H + 2 * Hm + 2 * Hm2), st>>>(emb, dlogit, pm, py1, py2, demb, w.Wg, pd1,
                                                                       pd2, dpre, dr, d.H);
  ++n;
  atb_f32(U, int(HU), dpre, d.H, gp(w.Wg), d.H, B, int(HU), d.H, st, gp(w.bg)); ++n;
  n += mlp_weight_grads(emb, d.H, B, d.Hm, d.Hm2, py1, py2, pd1, pd2, dlogit, gp(w.pW1), gp(w.pb1), gp(w.pWh),
                        gp(w.pbh), gp(w.pw2), gp(w.pb2), st);
  n += mlp_weight_grads(eb.vu, 2 * d.H, num_envs, d.Hm, d.Hm2, eb.vy1, eb.vy2, eb.vd1, eb.vd2, eb.vdout, gp(w.vW1),
                        gp(w.vb1), gp(w.vWh), gp(w.vbh), gp(w.vw2), gp(w.vb2), st);
  const int64_t ne = N * (d.H / 4);
  if (ne > 0) {
    const unsigned grid = unsigned(std::min<int64_t>((ne + 255) / 256, int64_t(kNumSMs) * 64));
    k_readout_bwd<<<grid, 256, 0, st>>>(dr, seg_id, dh, ne, d.H);
    ++n;
  }
  return n;
}

// One attention layer backwards: dh_out -> (dW, da_src, da_dst, db) and dh_in.  Z / scores hold the layer's
// forward transform of h_in; dz [N x H] and ds [2 N K] are scratch.
int launch_gat_layer_bwd(const Dims& d, const int32_t* rowptr, const int32_t* col, const void* Z, const float* scores,
                         const void* h_in, const void* h_out, const float* dh_out, float* dh_in, float* dz,
                         float* ds, void* dz_store, const LayerWeights& lw, float* gW, float* ga_src, float* ga_dst,
                         float* gb, int32_t N, cudaStream_t st) {
  if (N <= 0) return 0;
  const int H = d.H, K = d.K;
  cudaMemsetAsync(dz, 0, sizeof(float) * size_t(N) * H, st);
  cudaMemsetAsync(ds, 0, sizeof(float) * size_t(N) * K * 2, st);
  float* ds_src = ds;
  float* ds_dst = ds + size_t(N) * K;
  const size_t zrow = z_row_bytes(d);
  const int grid_rows = int(std::min<int64_t>((int64_t(N) + 7) / 8, int64_t(kNumSMs) * 8));
  const int grid_cols = int(std::min<int64_t>((int64_t(N) + 255) / 256, int64_t(kNumSMs) * 2));
  const int chunk = chunk_rows(N, 2048);
  dim3 g_atb(unsigned((H + 63) / 64), unsigned((H + 63) / 64), unsigned((N + chunk - 1) / chunk));
  dim3 g_gwt(unsigned((N + 63) / 64), unsigned((H + 63) / 64));
  // tensor-core products: about two waves of CTAs over the rows, chunks of a multiple of 32 rows, at least 512
  const int tiles = (H / 128) * (H / 128);
  const int want_chunks = std::max(1, 2 * kNumSMs / std::max(1, tiles));
  const int chunk_mma = std::max(512, int(((int64_t(N) + want_chunks - 1) / want_chunks + 31) & ~int64_t(31)));
  dim3 g_atb_mma(unsigned(H / 128), unsigned(H / 128), unsigned((N + chunk_mma - 1) / chunk_mma));
  const int row_tiles = (N + 127) / 128;
  const int gwt_tpc = int64_t(row_tiles) * (H / 128) >= int64_t(kGwtTiles) * 4 * kNumSMs ? kGwtTiles : 1;
  dim3 g_gwt_mma(unsigned((row_tiles + gwt_tpc - 1) / gwt_tpc) * unsigned(H / 128));
  const int NF = H / 32;
  const bool rows_kernels = (32 % K == 0) && (NF == 1 || NF == 2 || NF == 4 || NF == 8 || NF == 16);
  // bf16 models of hidden 128, 256 or 512 take both products on the tensor cores, from a bf16 copy of dz
  const bool mma = rows_kernels && d.dtype == XRL_BF16 && H % 128 == 0 && dz_store != nullptr;
  bf16* dzb = mma ? static_cast<bf16*>(dz_store) : nullptr;
#define BWD_ROWS(TY_, NF_)                                                                                     \
  do {                                                                                                         \
    k_aggregate_bwd_rows<TY_, NF_><<<grid_rows, 256, 0, st>>>(rowptr, col, zv, static_cast<const TY_*>(h_out), \
                                                              dh_out, dz, ds_src, ds_dst, gb, N, K);           \
    k_scores_bwd_rows<TY_, NF_><<<grid_rows, 256, 0, st>>>(zv, ds_src, ds_dst, lw.a_src, lw.a_dst, dz, dzb,    \
                                                           ga_src, ga_dst, N, K);                              \
  } while (0)
#define BWD_BODY(TY_)                                                                                          \
  do {                                                                                                         \
    ZView<TY_> zv;                                                                                             \
    zv.z = static_cast<const char*>(Z); zv.row_bytes = zrow;                                                   \
    zv.pairs = d.zmerged ? reinterpret_cast<const float2*>(static_cast<const char*>(Z) + size_t(H) * sizeof(TY_)) \
                         : reinterpret_cast<const float2*>(scores);                                          \
    zv.pair_stride = d.zmerged ? int(zrow / 8) : K;                                                            \
    if (rows_kernels) {                                                                                        \
      switch (NF) {                                                                                            \
        case 1: BWD_ROWS(TY_, 1); break;                                                                       \
        case 2: BWD_ROWS(TY_, 2); break;                                                                       \
        case 4: BWD_ROWS(TY_, 4); break;                                                                       \
        case 8: BWD_ROWS(TY_, 8); break;                                                                       \
        default: BWD_ROWS(TY_, 16); break;                                                                     \
      }                                                                                                        \
    } else {                                                                                                   \
      k_aggregate_bwd<TY_><<<grid_rows, 256, sizeof(float) * H, st>>>(                                         \
          rowptr, col, zv, static_cast<const TY_*>(h_out), dh_out, dz, ds_src, ds_dst, gb, N, H, K);           \
      k_scores_bwd<TY_><<<grid_cols, 256, sizeof(float) * 2 * H, st>>>(zv, ds_src, ds_dst, lw.a_src, lw.a_dst, \
                                                                       dz, ga_src, ga_dst, N, H, K);           \
    }                                                                                                          \
    if (mma) {                                                                                                 \
      k_atb_mma<<<g_atb_mma, 256, 0, st>>>(static_cast<const bf16*>(h_in), dzb, gW, N, H, chunk_mma);          \
      k_gwt_mma<<<g_gwt_mma, 256, 0, st>>>(dzb, static_cast<const bf16*>(lw.W), dh_in, N, H, gwt_tpc);                  \
    } else {                                                                                                   \
      k_atb<TY_><<<g_atb, 256, 0, st>>>(static_cast<const TY_*>(h_in), H, dz, H, gW, H, N, H, H, chunk, nullptr);       \
      k_gwt<TY_><<<g_gwt, 256, 0, st>>>(dz, static_cast<const TY_*>(lw.W), dh_in, N, H, H);                    \
    }                                                                                                          \
  } while (0)
  if (d.dtype == XRL_BF16) BWD_BODY(bf16); else BWD_BODY(float);
#undef BWD_ROWS
#undef BWD_BODY
  return 4;
}

// Eq. 6 in reverse keeps P copies of the one-hot block of W0's gradient ([T x H]) and a tile of R rows in shared
// memory: as many copies as threads share a column (at most 4), then the largest tile that still fits
static size_t embed_bwd_bytes(const Dims& d, int R, int P) {
  return sizeof(float) * (size_t(P) * d.T * d.H + size_t(R) * d.H + size_t(R) * 2 * kS) + sizeof(int32_t) * R;
}
static void embed_bwd_shape(const Dims& d, int* R, int* P) {
  constexpr size_t kCeiling = size_t(227) * 1024;
  *R = 0; *P = 1;
  for (int p = std::min(4, std::max(1, kEmbedBwdThreads / d.H)); p >= 1; --p)
    for (int r = 64; r >= 16; r >>= 1)
      if (embed_bwd_bytes(d, r, p) <= kCeiling) { *R = r; *P = p; return; }
  if (embed_bwd_bytes(d, 8, 1) <= kCeiling) *R = 8;
}
size_t embed_bwd_smem_bytes(const Dims& d) {
  int R, P;
  embed_bwd_shape(d, &R, &P);
  return embed_bwd_bytes(d, std::max(R, 8), P);
}

int launch_embed_bwd(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op, const void* shape,
                     const void* eattr, const void* h0, const float* dh0, float* xs, float* gW0, float* gb0, int32_t N,
                     cudaStream_t st) {
  if (N <= 0) return 0;
  int R, P;
  embed_bwd_shape(d, &R, &P);
  if (R == 0) return -1;
  const size_t smem = embed_bwd_bytes(d, R, P);
  const int grid = int(std::min<int64_t>((int64_t(N) + R - 1) / R, int64_t(kNumSMs)));
  const unsigned grid_x = unsigned((int64_t(N) + 255) / 256);
  // the opt-in is the kernel's ceiling for every later launch: ask for all an SM has, once per device
  constexpr int kSmemCeiling = 227 * 1024;
  if (d.dtype == XRL_BF16) {
    static bool attr[64] = {};
    if (!ensure_dynamic_smem(k_embed_bwd<bf16>, kSmemCeiling, attr)) return -1;
    k_embed_inputs<bf16><<<grid_x, 256, 0, st>>>(rowptr, col, static_cast<const bf16*>(shape),
                                                 static_cast<const bf16*>(eattr), xs, N);
    k_embed_bwd<bf16><<<grid, kEmbedBwdThreads, smem, st>>>(xs, op, static_cast<const bf16*>(h0), dh0, gW0, gb0, N,
                                                            d.H, d.T, R, P);
  } else {
    static bool attr[64] = {};
    if (!ensure_dynamic_smem(k_embed_bwd<float>, kSmemCeiling, attr)) return -1;
    k_embed_inputs<float><<<grid_x, 256, 0, st>>>(rowptr, col, static_cast<const float*>(shape),
                                                  static_cast<const float*>(eattr), xs, N);
    k_embed_bwd<float><<<grid, kEmbedBwdThreads, smem, st>>>(xs, op, static_cast<const float*>(h0), dh0, gW0, gb0, N,
                                                             d.H, d.T, R, P);
  }
  return 2;
}

}  // namespace xrl

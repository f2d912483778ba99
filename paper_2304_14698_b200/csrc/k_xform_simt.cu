// Dense node transform of a graph-attention layer, Z = h W (paper Eq. 7, the "W h_j" term), on
// the CUDA cores with fp32 accumulation.  This is the path for fp32 storage (whose tolerance a
// single-pass reduced-precision tensor-core product cannot guarantee) and for hidden sizes the
// tensor-core kernel is not built for.  The attention half-scores are taken from the accumulators in the
// kernel's last step when one tile spans all H columns, the storage is fp32 and a head is 4, 8, ... 128 columns
// wide (SCORES); otherwise from Z by k_scores.
#include "xrl_internal.cuh"

namespace xrl {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

// Half-scores of one row's 4-column group held by this thread: partial dot products with the attention
// vectors, summed over the `g` consecutive lanes that hold the same head of the same row (g a power of two
// <= 16; those lanes differ in the low bits of the lane id only).  Every lane gets the sums.
__device__ __forceinline__ void head_partial(const float (&z)[4], const float* __restrict__ a_src,
                                             const float* __restrict__ a_dst, int c, int g, float& ss, float& sd) {
  const float4 s = __ldg(reinterpret_cast<const float4*>(a_src + c));
  const float4 t = __ldg(reinterpret_cast<const float4*>(a_dst + c));
  ss = fmaf(z[3], s.w, fmaf(z[2], s.z, fmaf(z[1], s.y, z[0] * s.x)));
  sd = fmaf(z[3], t.w, fmaf(z[2], t.z, fmaf(z[1], t.y, z[0] * t.x)));
  for (int o = 1; o < g; o <<= 1) {
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    sd += __shfl_xor_sync(0xFFFFFFFFu, sd, o);
  }
}

template <typename T, bool SCORES>
__global__ void __launch_bounds__(256)
k_xform_simt(const T* __restrict__ h, const T* __restrict__ W, T* __restrict__ Z, int H, int rows,
             const float* __restrict__ a_src, const float* __restrict__ a_dst, float2* __restrict__ scores, int K) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  const int64_t row0 = int64_t(blockIdx.x) * BM;
  const int col0 = blockIdx.y * BN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int a_row = tid >> 2, a_k = (tid & 3) * 4;     // 64 rows x 16 k
  const int b_k = tid >> 4, b_c = (tid & 15) * 4;      // 16 k x 64 cols
  for (int k0 = 0; k0 < H; k0 += BK) {
    {
      const int64_t r = row0 + a_row;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int k = k0 + a_k + t;
        As[a_k + t][a_row] = (r < rows && k < H) ? to_float(h[size_t(r) * H + k]) : 0.f;
      }
      const int k = k0 + b_k;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int c = col0 + b_c + t;
        Bs[b_k][b_c + t] = (k < H && c < H) ? to_float(W[size_t(k) * H + c]) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t r = row0 + ty * 4 + i;
    if (SCORES) {                               // (every lane takes part in the shuffles)
      const int d = H / K, g = d >> 2, c = tx * 4;
      float ss = 0.f, sd = 0.f;
      const float z[4] = {acc[i][0], acc[i][1], acc[i][2], acc[i][3]};
      head_partial(z, a_src, a_dst, c < H ? c : 0, g, ss, sd);
      if (r < rows && c < H && (tx & (g - 1)) == 0) scores[size_t(r) * K + c / d] = make_float2(ss * kLog2e, sd * kLog2e);
    }
    if (r >= rows) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = col0 + tx * 4 + j;
      if (c < H) Z[size_t(r) * H + c] = T(acc[i][j]);
    }
  }
}

// Larger register tile for batches with many rows: 128 x 128 outputs per CTA, 8 x 8 per thread (as two
// 4-wide column groups and two 4-high row groups so that the shared-memory reads are conflict-free
// 16-byte loads), K advanced 8 at a time with the next slice prefetched into registers.
constexpr int TM = 128, TN = 128, TK = 8;

template <typename T>
__device__ __forceinline__ void load4(const T* p, bool ok, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, bool ok, float (&v)[4]) {
  const float4 t = ok ? __ldg(reinterpret_cast<const float4*>(p)) : make_float4(0.f, 0.f, 0.f, 0.f);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <>
__device__ __forceinline__ void load4<bf16>(const bf16* p, bool ok, float (&v)[4]) {
  const uint2 t = ok ? __ldg(reinterpret_cast<const uint2*>(p)) : make_uint2(0u, 0u);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
}

template <typename T, bool SCORES>
__global__ void __launch_bounds__(256)
k_xform_simt128(const T* __restrict__ h, const T* __restrict__ W, T* __restrict__ Z, int H, int rows,
                const float* __restrict__ a_src, const float* __restrict__ a_dst, float2* __restrict__ scores, int K) {
  __shared__ __align__(16) float As[TK][TM];
  __shared__ __align__(16) float Bs[TK][TN];
  const int tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  const int64_t row0 = int64_t(blockIdx.x) * TM;
  const int col0 = blockIdx.y * TN;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  const int a_row = tid >> 1, a_k = (tid & 1) * 4;      // 128 rows x 8 k: one 4-vector per thread
  const int b_k = tid >> 5, b_c = (tid & 31) * 4;       // 8 k x 128 cols
  const bool a_ok = row0 + a_row < rows;
  const T* a_ptr = h + size_t(a_ok ? row0 + a_row : 0) * H + a_k;
  const bool b_ok = col0 + b_c < H;                     // H is a multiple of 4
  const T* b_ptr = W + size_t(b_k) * H + (b_ok ? col0 + b_c : 0);
  float ra[4], rb[4];
  load4<T>(a_ptr, a_ok, ra);
  load4<T>(b_ptr, b_ok, rb);
  for (int k0 = 0; k0 < H; k0 += TK) {
#pragma unroll
    for (int t = 0; t < 4; ++t) As[a_k + t][a_row] = ra[t];
    *reinterpret_cast<float4*>(&Bs[b_k][b_c]) = make_float4(rb[0], rb[1], rb[2], rb[3]);
    __syncthreads();
    if (k0 + TK < H) {                                    // next slice in flight during the arithmetic
      load4<T>(a_ptr + k0 + TK, a_ok, ra);
      load4<T>(b_ptr + size_t(k0 + TK) * H, b_ok, rb);
    }
#pragma unroll
    for (int k = 0; k < TK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int64_t r = row0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (SCORES) {                               // (every lane takes part in the shuffles)
      const int d = H / K;
      float ss[2], sd[2];
#pragma unroll
      for (int jg = 0; jg < 2; ++jg) {
        const int c = jg * 64 + tx * 4;
        const float z[4] = {acc[i][jg * 4], acc[i][jg * 4 + 1], acc[i][jg * 4 + 2], acc[i][jg * 4 + 3]};
        head_partial(z, a_src, a_dst, c < H ? c : 0, d >= 64 ? 16 : (d >> 2), ss[jg], sd[jg]);   // (columns >= H hold 0)
      }
      if (r < rows) {
        if (d == 128) {                         // one head over both column groups
          if (tx == 0) scores[size_t(r) * K] = make_float2((ss[0] + ss[1]) * kLog2e, (sd[0] + sd[1]) * kLog2e);
        } else {
          const int g = d >= 64 ? 16 : (d >> 2);
#pragma unroll
          for (int jg = 0; jg < 2; ++jg) {
            const int c = jg * 64 + tx * 4;
            if (c < H && (tx & (g - 1)) == 0) scores[size_t(r) * K + c / d] = make_float2(ss[jg] * kLog2e, sd[jg] * kLog2e);
          }
        }
      }
    }
    if (r >= rows) continue;
#pragma unroll
    for (int jg = 0; jg < 2; ++jg) {
      const int c = col0 + jg * 64 + tx * 4;
      if (c >= H) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) Z[size_t(r) * H + c + j] = T(acc[i][jg * 4 + j]);
    }
  }
}

}  // namespace

// SCORES variant: fp32 storage, one tile across all H columns, heads 4 ... 128 columns wide (a power of two)
static bool fuse_scores(const Dims& d, int tile_cols, const float* scores) {
  if (d.dtype != XRL_FP32 || d.zmerged || scores == nullptr || d.H > tile_cols || (d.H & 3) || d.K < 1 || d.H % d.K) return false;
  const int w = d.H / d.K;
  return w >= 4 && w <= tile_cols && (w & (w - 1)) == 0;
}

int launch_xform_simt(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
                      Window win, cudaStream_t st) {
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  if (rows <= 0) return 0;
  const size_t off = size_t(win.row_begin - win.win_base) * d.H;
  float2* sc = reinterpret_cast<float2*>(scores) + size_t(win.row_begin - win.win_base) * d.K;
  if (rows >= 8192) {
    dim3 g128(unsigned((rows + TM - 1) / TM), unsigned((d.H + TN - 1) / TN));
    if (d.dtype == XRL_BF16) {
      k_xform_simt128<bf16, false><<<g128, 256, 0, st>>>(static_cast<const bf16*>(h) + off,
                                                         static_cast<const bf16*>(lw.W),
                                                         static_cast<bf16*>(Z) + off, d.H, int(rows), nullptr, nullptr,
                                                         nullptr, d.K);
    } else if (fuse_scores(d, TN, scores)) {
      k_xform_simt128<float, true><<<g128, 256, 0, st>>>(static_cast<const float*>(h) + off,
                                                         static_cast<const float*>(lw.W),
                                                         static_cast<float*>(Z) + off, d.H, int(rows), lw.a_src, lw.a_dst,
                                                         sc, d.K);
      return 1;
    } else {
      k_xform_simt128<float, false><<<g128, 256, 0, st>>>(static_cast<const float*>(h) + off,
                                                          static_cast<const float*>(lw.W),
                                                          static_cast<float*>(Z) + off, d.H, int(rows), nullptr, nullptr,
                                                          nullptr, d.K);
    }
    return 1 + launch_scores(d, Z, lw, scores, win, st);
  }
  dim3 grid(unsigned((rows + BM - 1) / BM), unsigned((d.H + BN - 1) / BN));
  if (d.dtype == XRL_BF16) {
    k_xform_simt<bf16, false><<<grid, 256, 0, st>>>(static_cast<const bf16*>(h) + off,
                                                   static_cast<const bf16*>(lw.W),
                                                   static_cast<bf16*>(Z) + off, d.H, int(rows), nullptr, nullptr, nullptr,
                                                   d.K);
  } else if (fuse_scores(d, BN, scores)) {
    k_xform_simt<float, true><<<grid, 256, 0, st>>>(static_cast<const float*>(h) + off,
                                                   static_cast<const float*>(lw.W),
                                                   static_cast<float*>(Z) + off, d.H, int(rows), lw.a_src, lw.a_dst, sc,
                                                   d.K);
    return 1;
  } else {
    k_xform_simt<float, false><<<grid, 256, 0, st>>>(static_cast<const float*>(h) + off,
                                                    static_cast<const float*>(lw.W),
                                                    static_cast<float*>(Z) + off, d.H, int(rows), nullptr, nullptr,
                                                    nullptr, d.K);
  }
  return 1 + launch_scores(d, Z, lw, scores, win, st);
}

}  // namespace xrl

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


// ---- fp32 storage, many rows: the product on the tensor cores with every operand split in two ----------------
// x = hi + lo with hi = tf32(x) and lo = tf32(x - hi); Z = sum hi_a hi_b + hi_a lo_b + lo_a hi_b in fp32
// accumulators (mma.sync m16n8k8, the small terms first): the dropped lo_a lo_b term is below 2^-22 of the
// product, i.e. the result is as good as an fp32 FMA chain in another order.  CTA tile 128 rows x 128 columns,
// 8 warps as 4 (rows) x 2 (columns), warp tile 32 x 64 = 2 x 8 MMA tiles; K advanced 16 at a time; both splits of a
// slice are made once, when it is written to shared memory (stored k-major: fragment reads are conflict-free
// with a row stride of 136 words).  Half-scores from the accumulators when a head is 8 ... 64 columns wide.
constexpr int XM = 128, XN = 128, XK = 16, XS = 136;

__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

template <bool SCORES>
__global__ void __launch_bounds__(256, 2)
k_xform_tf32x3(const float* __restrict__ h, const float* __restrict__ W, float* __restrict__ Z, int H, int rows,
               const float* __restrict__ a_src, const float* __restrict__ a_dst, float2* __restrict__ scores, int K) {
  extern __shared__ __align__(16) uint32_t xs[];          // A hi, A lo, B hi, B lo: each [XK][XS]
  uint32_t* Ah = xs;
  uint32_t* Al = Ah + XK * XS;
  uint32_t* Bh = Al + XK * XS;
  uint32_t* Bl = Bh + XK * XS;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int wm = (warp >> 1) * 32, wn = (warp & 1) * 64;  // the warp's tile inside the CTA tile
  const int64_t row0 = int64_t(blockIdx.x) * XM;
  const int col0 = blockIdx.y * XN;
  float acc[2][8][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  // loads of one slice: A 128 rows x 16 k = 512 float4 (two per thread), B 16 k x 128 columns = 512 float4
  const int a_row = tid >> 2, a_k = (tid & 3) * 4;        // and a_row + 64
  const int b_k = tid >> 5, b_c = (tid & 31) * 4;         // and b_k + 8
  const bool a_ok0 = row0 + a_row < rows, a_ok1 = row0 + a_row + 64 < rows;
  const bool b_ok = col0 + b_c < H;                       // H is a multiple of 4
  const float* a_p0 = h + size_t(a_ok0 ? row0 + a_row : 0) * H + a_k;
  const float* a_p1 = h + size_t(a_ok1 ? row0 + a_row + 64 : 0) * H + a_k;
  const float* b_p = W + size_t(b_k) * H + (b_ok ? col0 + b_c : 0);
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 ra0 = a_ok0 ? __ldg(reinterpret_cast<const float4*>(a_p0)) : zero4;
  float4 ra1 = a_ok1 ? __ldg(reinterpret_cast<const float4*>(a_p1)) : zero4;
  float4 rb0 = b_ok ? __ldg(reinterpret_cast<const float4*>(b_p)) : zero4;
  float4 rb1 = b_ok ? __ldg(reinterpret_cast<const float4*>(b_p + size_t(8) * H)) : zero4;

  auto split_store = [&](uint32_t* hi, uint32_t* lo, int idx, float x) {
    const uint32_t hb = to_tf32(x);
    hi[idx] = hb;
    lo[idx] = to_tf32(x - __uint_as_float(hb));
  };
  for (int k0 = 0; k0 < H; k0 += XK) {
    {
      const float a0[4] = {ra0.x, ra0.y, ra0.z, ra0.w}, a1[4] = {ra1.x, ra1.y, ra1.z, ra1.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        split_store(Ah, Al, (a_k + e) * XS + a_row, a0[e]);
        split_store(Ah, Al, (a_k + e) * XS + a_row + 64, a1[e]);
      }
      const float b0[4] = {rb0.x, rb0.y, rb0.z, rb0.w}, b1[4] = {rb1.x, rb1.y, rb1.z, rb1.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        split_store(Bh, Bl, b_k * XS + b_c + e, b0[e]);
        split_store(Bh, Bl, (b_k + 8) * XS + b_c + e, b1[e]);
      }
    }
    __syncthreads();
    if (k0 + XK < H) {                                    // next slice in flight during the arithmetic
      ra0 = a_ok0 ? __ldg(reinterpret_cast<const float4*>(a_p0 + k0 + XK)) : zero4;
      ra1 = a_ok1 ? __ldg(reinterpret_cast<const float4*>(a_p1 + k0 + XK)) : zero4;
      rb0 = b_ok ? __ldg(reinterpret_cast<const float4*>(b_p + size_t(k0 + XK) * H)) : zero4;
      rb1 = b_ok ? __ldg(reinterpret_cast<const float4*>(b_p + size_t(k0 + XK + 8) * H)) : zero4;
    }
#pragma unroll
    for (int ks = 0; ks < XK; ks += 8) {
      uint32_t ah[2][4], al[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int r = wm + i * 16 + g;
        // fragment of a 16 x 8 tile: (row g, k t), (row g + 8, k t), (row g, k t + 4), (row g + 8, k t + 4)
        ah[i][0] = Ah[(ks + t) * XS + r];     ah[i][1] = Ah[(ks + t) * XS + r + 8];
        ah[i][2] = Ah[(ks + t + 4) * XS + r]; ah[i][3] = Ah[(ks + t + 4) * XS + r + 8];
        al[i][0] = Al[(ks + t) * XS + r];     al[i][1] = Al[(ks + t) * XS + r + 8];
        al[i][2] = Al[(ks + t + 4) * XS + r]; al[i][3] = Al[(ks + t + 4) * XS + r + 8];
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int c = wn + j * 8 + g;
        // fragment of an 8 x 8 tile: (k t, column g), (k t + 4, column g)
        const uint32_t bh[2] = {Bh[(ks + t) * XS + c], Bh[(ks + t + 4) * XS + c]};
        const uint32_t bl[2] = {Bl[(ks + t) * XS + c], Bl[(ks + t + 4) * XS + c]};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          mma_tf32(acc[i][j], al[i], bh);
          mma_tf32(acc[i][j], ah[i], bl);
          mma_tf32(acc[i][j], ah[i], bh);
        }
      }
    }
    __syncthreads();
  }
  // accumulator of an MMA tile: (row g, columns 2t, 2t + 1), (row g + 8, columns 2t, 2t + 1)
#pragma unroll
  for (int i = 0; i < 2; ++i) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int64_t r = row0 + wm + i * 16 + g + half * 8;
      if (SCORES) {                             // (every lane takes part in the shuffles)
        const int d = H / K, tiles = d >> 3;    // MMA tiles per head: 1, 2, 4 or 8
        float ss = 0.f, sd = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int c = col0 + wn + j * 8 + 2 * t;
          const int cc = c < H ? c : 0;         // (columns >= H hold 0)
          const float2 s = __ldg(reinterpret_cast<const float2*>(a_src + cc));
          const float2 u = __ldg(reinterpret_cast<const float2*>(a_dst + cc));
          ss = fmaf(acc[i][j][2 * half + 1], s.y, fmaf(acc[i][j][2 * half], s.x, ss));
          sd = fmaf(acc[i][j][2 * half + 1], u.y, fmaf(acc[i][j][2 * half], u.x, sd));
          if (((j + 1) & (tiles - 1)) == 0) {   // the head ends with this tile
            ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1); sd += __shfl_xor_sync(0xFFFFFFFFu, sd, 1);
            ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2); sd += __shfl_xor_sync(0xFFFFFFFFu, sd, 2);
            if (t == 0 && r < rows && c < H) scores[size_t(r) * K + c / d] = make_float2(ss * kLog2e, sd * kLog2e);
            ss = 0.f; sd = 0.f;
          }
        }
      }
      if (r >= rows) continue;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int c = col0 + wn + j * 8 + 2 * t;
        if (c < H) *reinterpret_cast<float2*>(Z + size_t(r) * H + c) = make_float2(acc[i][j][2 * half], acc[i][j][2 * half + 1]);
      }
    }
  }
}

}  // namespace

// SCORES variant: fp32 storage, one tile across all H columns, heads 4 ... 128 columns wide (a power of two)
static bool fuse_scores(const Dims& d, const LayerWeights& lw, int tile_cols, const float* scores, int min_width = 4) {
  if (d.dtype != XRL_FP32 || d.zmerged || scores == nullptr || d.H > tile_cols || (d.H & 3) || d.K < 1 || d.H % d.K) return false;
  if ((reinterpret_cast<uintptr_t>(lw.a_src) | reinterpret_cast<uintptr_t>(lw.a_dst)) & 15) return false;   // vector loads
  const int w = d.H / d.K;
  return w >= min_width && w <= tile_cols && (w & (w - 1)) == 0;
}

int launch_xform_simt(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
                      Window win, cudaStream_t st) {
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  if (rows <= 0) return 0;
  const size_t off = size_t(win.row_begin - win.win_base) * d.H;
  float2* sc = reinterpret_cast<float2*>(scores) + size_t(win.row_begin - win.win_base) * d.K;
  if (rows >= 8192 && d.dtype == XRL_FP32 && d.H % XK == 0) {
    // fp32 storage: split operands on the tensor cores
    dim3 gx(unsigned((rows + XM - 1) / XM), unsigned((d.H + XN - 1) / XN));
    const size_t smem = sizeof(uint32_t) * 4 * XK * XS;
    const int w = d.H / d.K;
    if (fuse_scores(d, lw, XN, scores, 8) && w <= 64) {
      k_xform_tf32x3<true><<<gx, 256, smem, st>>>(static_cast<const float*>(h) + off, static_cast<const float*>(lw.W),
                                                 static_cast<float*>(Z) + off, d.H, int(rows), lw.a_src, lw.a_dst, sc, d.K);
      return 1;
    }
    k_xform_tf32x3<false><<<gx, 256, smem, st>>>(static_cast<const float*>(h) + off, static_cast<const float*>(lw.W),
                                                static_cast<float*>(Z) + off, d.H, int(rows), nullptr, nullptr, nullptr,
                                                d.K);
    return 1 + launch_scores(d, Z, lw, scores, win, st);
  }
  if (rows >= 8192) {
    dim3 g128(unsigned((rows + TM - 1) / TM), unsigned((d.H + TN - 1) / TN));
    if (d.dtype == XRL_BF16) {
      k_xform_simt128<bf16, false><<<g128, 256, 0, st>>>(static_cast<const bf16*>(h) + off,
                                                         static_cast<const bf16*>(lw.W),
                                                         static_cast<bf16*>(Z) + off, d.H, int(rows), nullptr, nullptr,
                                                         nullptr, d.K);
    } else if (fuse_scores(d, lw, TN, scores)) {
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
  } else if (fuse_scores(d, lw, BN, scores)) {
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

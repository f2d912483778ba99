// Dense node transform of a graph-attention layer, Z = h W (paper Eq. 7, the "W h_j" term), on
// the CUDA cores with fp32 accumulation.  This is the path for fp32 storage (whose tolerance a
// single-pass reduced-precision tensor-core product cannot guarantee) and for hidden sizes the
// tensor-core kernel is not built for.  The attention half-scores are taken from Z by k_scores.
#include "xrl_internal.cuh"

namespace xrl {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__global__ void __launch_bounds__(256)
k_xform_simt(const T* __restrict__ h, const T* __restrict__ W, T* __restrict__ Z, int H, int rows) {
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
    if (r >= rows) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = col0 + tx * 4 + j;
      if (c < H) Z[size_t(r) * H + c] = T(acc[i][j]);
    }
  }
}

}  // namespace

int launch_xform_simt(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
                      Window win, cudaStream_t st) {
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  if (rows <= 0) return 0;
  const size_t off = size_t(win.row_begin - win.win_base) * d.H;
  dim3 grid(unsigned((rows + BM - 1) / BM), unsigned((d.H + BN - 1) / BN));
  if (d.dtype == XRL_BF16)
    k_xform_simt<bf16><<<grid, 256, 0, st>>>(static_cast<const bf16*>(h) + off,
                                            static_cast<const bf16*>(lw.W),
                                            static_cast<bf16*>(Z) + off, d.H, int(rows));
  else
    k_xform_simt<float><<<grid, 256, 0, st>>>(static_cast<const float*>(h) + off,
                                             static_cast<const float*>(lw.W),
                                             static_cast<float*>(Z) + off, d.H, int(rows));
  return 1 + launch_scores(d, Z, lw, scores, win, st);
}

}  // namespace xrl

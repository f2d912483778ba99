// Dense node transform of a graph-attention layer on the 5th-generation tensor cores:
// Z = h W (paper Eq. 7, the "W h_j" term) for bf16 storage, fp32 accumulation in tensor memory,
// with the per-head attention half-scores s_src = a_src . Z_k, s_dst = a_dst . Z_k taken from the
// fp32 accumulators in the epilogue.
//
// One persistent CTA per SM.  W^T (the K-major B operand, H x H bf16) stays resident in shared
// memory; 128-row tiles of h stream through a ring of TMA-loaded, 128-byte-swizzled stages; one
// thread issues tcgen05.mma (M = 128, N = H, K = 16) into one of two accumulator buffers in
// tensor memory; four epilogue warps read the accumulators back (tcgen05.ld), form the
// half-scores, round Z to bf16 into a swizzled staging tile and hand it to a TMA store.
// The op moves 2 H b bytes per node against 2 H^2 flops: it is bound by HBM, not by the tensor
// pipe, so the design goal is to keep loads and stores streaming.
//
// Every wait on an mbarrier is bounded; on expiry the kernel records XRL_ERR_TIMEOUT, drains its
// own copies in flight, frees its tensor memory and returns.
#include "xrl_xform_umma.cuh"

namespace xrl {

using namespace umma;
using namespace xform;

namespace {

constexpr int kThreads = 192;           // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue

template <int H>
__global__ void __launch_bounds__(kThreads, 1)
k_xform_umma(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
             const __grid_constant__ CUtensorMap map_z, const float* __restrict__ a_src,
             const float* __restrict__ a_dst, float2* __restrict__ scores, int score_stride,
             int rows, int K, int32_t* status) {
  using C = Cfg<H>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t base = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = (rows + BM - 1) / BM;

  if ((base & 1023u) != 0) {               // the swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) raise(status, XRL_ERR_UNSUPPORTED);
    return;
  }
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_TMEM);
  float* avec = reinterpret_cast<float*>(smem + C::OFF_AVEC);

  if (threadIdx.x == 0) {
    tmem_slot[1] = 0;
    init_barriers<H>(base);
  }
  // attention vectors pre-multiplied by log2(e): the half-scores are consumed by an exp2 softmax
  for (int t = threadIdx.x; t < H; t += kThreads) { avec[t] = a_src[t] * kLog2e; avec[H + t] = a_dst[t] * kLog2e; }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(uint32_t(C::TMEM_COLS)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---- TMA producer ---------------------------------------------------------------------------
    if (lane == 0) {
      load_w<H>(base, &map_w);
      uint32_t it = 0;
      if (!produce_tiles<H>(base, &map_h, blockIdx.x, gridDim.x, num_tiles, it)) {
        raise(status, XRL_ERR_TIMEOUT);
        drain_producer<H>(base, it, 0);
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------
    if (lane == 0) {
      uint32_t it = 0, lt = 0;
      if (!mma_tiles<H>(base, tmem_base, blockIdx.x, gridDim.x, num_tiles, it, lt, 0)) raise(status, XRL_ERR_TIMEOUT);
    }
  } else {
    // ---- epilogue: 4 warps ------------------------------------------------------------------------
    uint32_t lt = 0;
    epilogue_tiles<H>(smem, base, tmem_base, &map_z, scores, score_stride, rows, K, blockIdx.x, gridDim.x,
                      num_tiles, lt, threadIdx.x == 64, status);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"(uint32_t(C::TMEM_COLS)) : "memory");
  }
}

template <int H>
int launch_h(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
             Window win, int32_t* status, cudaStream_t st) {
  using C = Cfg<H>;
  static bool attr_set[64] = {};
  if (!ensure_dynamic_smem(k_xform_umma<H>, C::SMEM_BYTES, attr_set)) return -1;
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  const size_t off = size_t(win.row_begin - win.win_base);
  const bf16* hp = static_cast<const bf16*>(h) + off * H;
  const size_t zrow = z_row_bytes(d);                    // H * 2, or H * 2 + 8 K when the pairs follow the row
  char* zp = static_cast<char*>(Z) + off * zrow;
  float2* sc = d.zmerged ? reinterpret_cast<float2*>(zp + size_t(H) * 2)
                         : reinterpret_cast<float2*>(scores) + off * d.K;
  const int sc_stride = d.zmerged ? int(zrow / 8) : d.K;
  CUtensorMap mh, mw, mz;
  if (!make_map(&mh, hp, uint64_t(rows), H, BM) || !make_map(&mw, lw.Wt, H, H, H) ||
      !make_map(&mz, zp, uint64_t(rows), H, BM, zrow))
    return -1;
  const int tiles = int((rows + BM - 1) / BM);
  const int grid = tiles < kNumSMs ? tiles : kNumSMs;
  k_xform_umma<H><<<grid, kThreads, C::SMEM_BYTES, st>>>(mh, mw, mz, lw.a_src, lw.a_dst, sc, sc_stride,
                                                         int(rows), d.K, status);
  return 1;
}

}  // namespace

bool xform_umma_supported(const Dims& d) {
  return d.dtype == XRL_BF16 && (d.H == 128 || d.H == 256) && encode_fn() != nullptr;
}

// Returns the number of kernels launched, or -1 if the tensor maps could not be built.
int launch_xform_umma(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
                      Window win, int32_t* status, cudaStream_t st) {
  if (int64_t(win.row_end) - win.row_begin <= 0) return 0;
  if (d.H == 256) return launch_h<256>(d, h, lw, Z, scores, win, status, st);
  return launch_h<128>(d, h, lw, Z, scores, win, status, st);
}

}  // namespace xrl

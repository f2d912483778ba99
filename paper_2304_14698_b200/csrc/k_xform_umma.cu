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
#include "xrl_umma.cuh"

namespace xrl {

using namespace umma;

namespace {

constexpr int BM = 128;                 // rows per tile (UMMA M)
constexpr int STAGE_BYTES = BM * 128;   // one A stage / one output staging tile: 128 rows x 128 B
constexpr int kThreads = 192;           // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue

template <int H> struct Cfg {
  static constexpr int KC = H / KCH;                    // K chunks (= output column chunks)
  static constexpr int W_CHUNK_BYTES = H * 128;         // N rows x 128 B
  static constexpr int W_BYTES = KC * W_CHUNK_BYTES;
  static constexpr int STAGES = (H == 256) ? 4 : 8;
  static constexpr int TMEM_COLS = 2 * H;               // two fp32 accumulators of N = H columns
  static constexpr int OFF_A = W_BYTES;
  static constexpr int OFF_OUT = OFF_A + STAGES * STAGE_BYTES;
  static constexpr int OFF_AVEC = OFF_OUT + 2 * STAGE_BYTES;
  static constexpr int OFF_BAR = OFF_AVEC + 2 * H * 4;
  static constexpr int NUM_BARS = 1 + 2 * STAGES + 4;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;   // [0] TMEM base address, [1] abort flag
  static constexpr int SMEM_BYTES = OFF_TMEM + 16;
};

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
  const uint32_t bar0 = base + C::OFF_BAR;
  const uint32_t bar_w = bar0;
  auto bar_a_full = [&](int s) { return bar0 + 8u * (1 + s); };
  auto bar_a_empty = [&](int s) { return bar0 + 8u * (1 + C::STAGES + s); };
  auto bar_acc_full = [&](int b) { return bar0 + 8u * (1 + 2 * C::STAGES + b); };
  auto bar_acc_empty = [&](int b) { return bar0 + 8u * (1 + 2 * C::STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_TMEM);
  float* avec = reinterpret_cast<float*>(smem + C::OFF_AVEC);

  if (threadIdx.x == 0) {
    tmem_slot[1] = 0;
    mbar_init(bar_w, 1);
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(bar_a_full(s), 1); mbar_init(bar_a_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_acc_full(b), 1); mbar_init(bar_acc_empty(b), 128); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
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
      bool ok = true;
      mbar_expect_tx(bar_w, C::W_BYTES);
      for (int kc = 0; kc < C::KC; ++kc)
        tma_load_2d(base + kc * C::W_CHUNK_BYTES, &map_w, kc * KCH, 0, bar_w);
      uint32_t it = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        for (int kc = 0; kc < C::KC; ++kc, ++it) {
          const int s = it % C::STAGES;
          const uint32_t round = it / C::STAGES;
          if (round > 0 && !mbar_wait(bar_a_empty(s), (round - 1) & 1)) { ok = false; break; }
          mbar_expect_tx(bar_a_full(s), STAGE_BYTES);
          tma_load_2d(base + C::OFF_A + s * STAGE_BYTES, &map_h, kc * KCH, tile * BM, bar_a_full(s));
        }
      }
      if (!ok) {
        raise(status, XRL_ERR_TIMEOUT);
        // let the loads already issued land before the CTA's shared memory goes away
        const uint32_t first = it > uint32_t(C::STAGES) ? it - C::STAGES : 0;
        for (uint32_t j = first; j < it; ++j) mbar_wait(bar_a_full(j % C::STAGES), (j / C::STAGES) & 1);
        mbar_wait(bar_w, 0);
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(H >> 3) << 17) |
                                 (uint32_t(BM >> 4) << 24);   // fp32 accum, bf16 x bf16, K-major both
      bool ok = mbar_wait(bar_w, 0);
      tc_fence_after();
      uint32_t it = 0, lt = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
        const int buf = lt & 1;
        const uint32_t use = lt >> 1;
        if (use > 0 && !mbar_wait(bar_acc_empty(buf), (use - 1) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + uint32_t(buf * H);
        for (int kc = 0; kc < C::KC; ++kc, ++it) {
          const int s = it % C::STAGES;
          if (!mbar_wait(bar_a_full(s), (it / C::STAGES) & 1)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = base + C::OFF_A + s * STAGE_BYTES;
          const uint32_t b_addr = base + kc * C::W_CHUNK_BYTES;
#pragma unroll
          for (int k = 0; k < KCH / 16; ++k)
            tc_mma(tmem_d, smem_desc(a_addr + k * 32), smem_desc(b_addr + k * 32), idesc,
                   (kc | k) != 0 ? 1u : 0u);
          tc_commit(bar_a_empty(s));        // the stage is free once these MMAs have read it
        }
        if (!ok) break;
        tc_commit(bar_acc_full(buf));       // the accumulator is complete
      }
      if (!ok) raise(status, XRL_ERR_TIMEOUT);
    }
  } else {
    // ---- epilogue: 4 warps, warp q reads tensor-memory lanes [32 q, 32 q + 32) --------------------
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const bool leader = (threadIdx.x == 64);
    const int d = H / K;                         // head width, a multiple of 8
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint32_t lt = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++lt) {
      const int buf = lt & 1;
      // one lane per warp waits; the four warps agree on the outcome before touching a barrier
      uint32_t okw = 1;
      if (lane == 0) okw = mbar_wait(bar_acc_full(buf), (lt >> 1) & 1) ? 1u : 0u;
      okw = __shfl_sync(0xFFFFFFFFu, okw, 0);
      if (!okw && lane == 0) { *abort_flag = 1; raise(status, XRL_ERR_TIMEOUT); }
      epi_barrier();
      if (*abort_flag) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(buf * H);
      const int64_t grow = int64_t(tile) * BM + row_in_tile;
      const bool live = grow < rows;
      float ss = 0.f, sd = 0.f;
      int head = 0, left = d;                    // columns left in the current head
      for (int c = 0; c < C::KC; ++c) {          // 64 output columns per chunk
        uint32_t v[2][32];
        tc_ld32(taddr + c * 64, v[0]);
        tc_ld32(taddr + c * 64 + 32, v[1]);
        tc_wait_ld();
        // half-scores from the fp32 accumulators, eight columns at a time
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const float4* as = reinterpret_cast<const float4*>(avec + c * 64 + g * 8);
          const float4* ad = reinterpret_cast<const float4*>(avec + H + c * 64 + g * 8);
          const float4 s0 = as[0], s1 = as[1], d0 = ad[0], d1 = ad[1];
          const uint32_t* z = &v[g >> 2][(g & 3) * 8];
          ss = fmaf(__uint_as_float(z[0]), s0.x, ss); sd = fmaf(__uint_as_float(z[0]), d0.x, sd);
          ss = fmaf(__uint_as_float(z[1]), s0.y, ss); sd = fmaf(__uint_as_float(z[1]), d0.y, sd);
          ss = fmaf(__uint_as_float(z[2]), s0.z, ss); sd = fmaf(__uint_as_float(z[2]), d0.z, sd);
          ss = fmaf(__uint_as_float(z[3]), s0.w, ss); sd = fmaf(__uint_as_float(z[3]), d0.w, sd);
          ss = fmaf(__uint_as_float(z[4]), s1.x, ss); sd = fmaf(__uint_as_float(z[4]), d1.x, sd);
          ss = fmaf(__uint_as_float(z[5]), s1.y, ss); sd = fmaf(__uint_as_float(z[5]), d1.y, sd);
          ss = fmaf(__uint_as_float(z[6]), s1.z, ss); sd = fmaf(__uint_as_float(z[6]), d1.z, sd);
          ss = fmaf(__uint_as_float(z[7]), s1.w, ss); sd = fmaf(__uint_as_float(z[7]), d1.w, sd);
          left -= 8;
          if (left == 0) {
            if (live) scores[grow * score_stride + head] = make_float2(ss, sd);
            ss = 0.f; sd = 0.f; ++head; left = d;
          }
        }
        // staging tile (c & 1) must no longer be read by the store issued two chunks ago
        if (leader) tma_wait_read<1>();
        epi_barrier();
        uint8_t* stage = smem + C::OFF_OUT + (c & 1) * STAGE_BYTES + row_in_tile * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {            // 16-byte chunk j of this row, swizzled by the row
          const uint32_t* z = &v[j >> 2][(j & 3) * 8];
          uint4 pk;
          pk.x = pack_bf16x2(__uint_as_float(z[0]), __uint_as_float(z[1]));
          pk.y = pack_bf16x2(__uint_as_float(z[2]), __uint_as_float(z[3]));
          pk.z = pack_bf16x2(__uint_as_float(z[4]), __uint_as_float(z[5]));
          pk.w = pack_bf16x2(__uint_as_float(z[6]), __uint_as_float(z[7]));
          *reinterpret_cast<uint4*>(stage + ((j ^ (row_in_tile & 7)) << 4)) = pk;
        }
        fence_async_smem();
        epi_barrier();
        if (leader) {
          tma_store_2d(&map_z, base + C::OFF_OUT + (c & 1) * STAGE_BYTES, c * 64, tile * BM);
          tma_commit();
        }
      }
      tc_fence_before();
      mbar_arrive(bar_acc_empty(buf));           // 128 arrivals free the accumulator
    }
    if (leader) tma_wait_all();
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

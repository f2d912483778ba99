// Device code of the tensor-core node transform (paper Eq. 7, Z = h W with the per-head attention
// half-scores taken from the fp32 accumulators), shared by the kernel that runs one layer per launch
// and by the kernel that runs all layers of a small step in one launch: shared-memory layout and the
// three roles (TMA producer, MMA issuer, epilogue) as routines over a CTA's tiles.  The counters a
// role passes by reference carry the positions in the stage ring and in the accumulator pair from one
// call to the next, so that a role can be called once per layer on the same barriers.
#pragma once

#include "xrl_umma.cuh"

namespace xrl {
namespace xform {

using namespace umma;

constexpr int BM = 128;                 // rows per tile (UMMA M)
constexpr int STAGE_BYTES = BM * 128;   // one A stage / one output staging tile: 128 rows x 128 B

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

  __device__ static uint32_t bar_w(uint32_t base) { return base + OFF_BAR; }
  __device__ static uint32_t bar_a_full(uint32_t base, int s) { return base + OFF_BAR + 8u * (1 + s); }
  __device__ static uint32_t bar_a_empty(uint32_t base, int s) { return base + OFF_BAR + 8u * (1 + STAGES + s); }
  __device__ static uint32_t bar_acc_full(uint32_t base, int b) { return base + OFF_BAR + 8u * (1 + 2 * STAGES + b); }
  __device__ static uint32_t bar_acc_empty(uint32_t base, int b) {
    return base + OFF_BAR + 8u * (1 + 2 * STAGES + 2 + b);
  }
};

// One thread: barriers of the layout above (128 epilogue threads free an accumulator).
template <int H> __device__ __forceinline__ void init_barriers(uint32_t base) {
  using C = Cfg<H>;
  mbar_init(C::bar_w(base), 1);
  for (int s = 0; s < C::STAGES; ++s) { mbar_init(C::bar_a_full(base, s), 1); mbar_init(C::bar_a_empty(base, s), 1); }
  for (int b = 0; b < 2; ++b) { mbar_init(C::bar_acc_full(base, b), 1); mbar_init(C::bar_acc_empty(base, b), 128); }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_async_smem();
}

// One thread: W^T (K-major, H x H bf16) into the start of shared memory; completion on bar_w.
template <int H> __device__ __forceinline__ void load_w(uint32_t base, const CUtensorMap* map_w) {
  using C = Cfg<H>;
  mbar_expect_tx(C::bar_w(base), C::W_BYTES);
  for (int kc = 0; kc < C::KC; ++kc) tma_load_2d(base + kc * C::W_CHUNK_BYTES, map_w, kc * KCH, 0, C::bar_w(base));
}

// One thread: the A tiles first, first + step, ... < num_tiles through the stage ring.  False on a timeout.
template <int H>
__device__ __forceinline__ bool produce_tiles(uint32_t base, const CUtensorMap* map_h, int first, int step,
                                              int num_tiles, uint32_t& it) {
  using C = Cfg<H>;
  for (int tile = first; tile < num_tiles; tile += step) {
    for (int kc = 0; kc < C::KC; ++kc, ++it) {
      const int s = it % C::STAGES;
      const uint32_t round = it / C::STAGES;
      if (round > 0 && !mbar_wait(C::bar_a_empty(base, s), (round - 1) & 1)) return false;
      mbar_expect_tx(C::bar_a_full(base, s), STAGE_BYTES);
      tma_load_2d(base + C::OFF_A + s * STAGE_BYTES, map_h, kc * KCH, tile * BM, C::bar_a_full(base, s));
    }
  }
  return true;
}

// After a producer timeout: let the loads already issued land before the CTA's shared memory goes away.
template <int H> __device__ __forceinline__ void drain_producer(uint32_t base, uint32_t it, uint32_t w_parity) {
  using C = Cfg<H>;
  const uint32_t first = it > uint32_t(C::STAGES) ? it - C::STAGES : 0;
  for (uint32_t j = first; j < it; ++j) mbar_wait(C::bar_a_full(base, j % C::STAGES), (j / C::STAGES) & 1);
  mbar_wait(C::bar_w(base), w_parity);
}

// One thread: tcgen05.mma (M = 128, N = H, K = 16) over the same tiles, alternating between the two
// accumulators; waits for W (phase w_parity of bar_w) first.  False on a timeout.
template <int H>
__device__ __forceinline__ bool mma_tiles(uint32_t base, uint32_t tmem_base, int first, int step, int num_tiles,
                                          uint32_t& it, uint32_t& lt, uint32_t w_parity) {
  using C = Cfg<H>;
  constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(H >> 3) << 17) |
                             (uint32_t(BM >> 4) << 24);   // fp32 accum, bf16 x bf16, K-major both
  if (!mbar_wait(C::bar_w(base), w_parity)) return false;
  tc_fence_after();
  for (int tile = first; tile < num_tiles; tile += step, ++lt) {
    const int buf = lt & 1;
    const uint32_t use = lt >> 1;
    if (use > 0 && !mbar_wait(C::bar_acc_empty(base, buf), (use - 1) & 1)) return false;
    tc_fence_after();
    const uint32_t tmem_d = tmem_base + uint32_t(buf * H);
    for (int kc = 0; kc < C::KC; ++kc, ++it) {
      const int s = it % C::STAGES;
      if (!mbar_wait(C::bar_a_full(base, s), (it / C::STAGES) & 1)) return false;
      tc_fence_after();
      const uint32_t a_addr = base + C::OFF_A + s * STAGE_BYTES;
      const uint32_t b_addr = base + kc * C::W_CHUNK_BYTES;
#pragma unroll
      for (int k = 0; k < KCH / 16; ++k)
        tc_mma(tmem_d, smem_desc(a_addr + k * 32), smem_desc(b_addr + k * 32), idesc, (kc | k) != 0 ? 1u : 0u);
      tc_commit(C::bar_a_empty(base, s));       // the stage is free once these MMAs have read it
    }
    tc_commit(C::bar_acc_full(base, buf));      // the accumulator is complete
  }
  return true;
}

// The four epilogue warps (CTA warps 2..5; warp q = warp & 3 reads tensor-memory lanes [32 q, 32 q + 32)):
// per tile the half-scores from the fp32 accumulators, Z rounded to bf16 into a swizzled staging tile,
// TMA store.  `leader` is one of the 128 threads; it owns the stores and waits for them at the end.
// A timeout sets the abort word behind the tensor-memory slot and raises XRL_ERR_TIMEOUT.
template <int H>
__device__ __forceinline__ void epilogue_tiles(uint8_t* smem, uint32_t base, uint32_t tmem_base,
                                               const CUtensorMap* map_z, float2* __restrict__ scores,
                                               int score_stride, int rows, int K, int first, int step,
                                               int num_tiles, uint32_t& lt, bool leader, int32_t* status) {
  using C = Cfg<H>;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = warp & 3;
  const int row_in_tile = q * 32 + lane;
  const int d = H / K;                         // head width, a multiple of 8
  const float* avec = reinterpret_cast<const float*>(smem + C::OFF_AVEC);
  volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(smem + C::OFF_TMEM) + 1;
  for (int tile = first; tile < num_tiles; tile += step, ++lt) {
    const int buf = lt & 1;
    // one lane per warp waits; the four warps agree on the outcome before touching a barrier
    uint32_t okw = 1;
    if (lane == 0) okw = mbar_wait(C::bar_acc_full(base, buf), (lt >> 1) & 1) ? 1u : 0u;
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
        tma_store_2d(map_z, base + C::OFF_OUT + (c & 1) * STAGE_BYTES, c * 64, tile * BM);
        tma_commit();
      }
    }
    tc_fence_before();
    mbar_arrive(C::bar_acc_empty(base, buf));   // 128 arrivals free the accumulator
  }
  if (leader) tma_wait_all();
}

}  // namespace xform
}  // namespace xrl

// Device code of the TMA-gather attention kernel (paper Eq. 7: edge score, segment softmax, weighted
// aggregate), shared by the kernel that runs one layer per launch and by the kernel that runs all
// layers of a small step in one launch: per-warp ring layout, the packed fp32 arithmetic, and the
// routine in which one warp works through blocks of destination rows.
#pragma once

#include "xrl_umma.cuh"

namespace xrl {
namespace aggtma {

using namespace umma;

constexpr int BR = 32;           // destination rows per block at most (a launch may take 16 or 8)
constexpr int ITEMS = 160;       // list capacity, a multiple of 4

// One warp's shared memory.  G gather groups in flight, each of GQ gathers of four rows.
// MERGED: the rows of Z carry their K {s_src, s_dst} pairs behind the 512 feature bytes, so one gather
// per group brings both; otherwise the pairs come from a second gather into `sc`.
template <int K, bool MERGED, int G, int GQ> struct alignas(128) WarpSmem {
  static constexpr int GV = 4 * GQ;                          // vectors (rows) per group
  static constexpr int ROW = MERGED ? 512 + 8 * K : 512;     // bytes per gathered row
  uint8_t z[G][GV][ROW];         // the gathered rows of a group
  float2 sc[MERGED ? 1 : G][GV][K];  // their {s_src, s_dst} pairs (separate gather only)
  unsigned long long bar[G];
  int32_t rp[BR + 1];
  alignas(16) int32_t item[ITEMS + GV];
};

__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* map, int r0, int r1, int r2,
                                            int r3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(map), "r"(0), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 lds64(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lrelu(float x) { return fmaxf(x, 0.2f * x); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Bounded wait executed by every lane (each lane must observe the phase itself to see the data).
__device__ __forceinline__ bool wait_all_lanes(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < (1 << 20); ++it)
    if (mbar_try(bar, parity)) return true;
  return false;
}

// Two fp32 lanes per instruction (sm_100): acc = p * z + acc on register pairs.
struct F2 { unsigned long long v; };
__device__ __forceinline__ F2 make_f2(float lo, float hi) {
  F2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void split_f2(F2 a, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v));
}
__device__ __forceinline__ void fma2(F2& acc, F2 p, F2 z) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc.v) : "l"(p.v), "l"(z.v));
}
__device__ __forceinline__ void mul2(F2& acc, F2 p) {
  asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(acc.v) : "l"(p.v));
}
__device__ __forceinline__ void add2(F2& acc, F2 x) {
  asm("add.rn.f32x2 %0, %0, %1;" : "+l"(acc.v) : "l"(x.v));
}

// Per-lane accumulator of one destination row: NP register pairs.
template <int VEC> struct Acc { F2 a[VEC / 2]; };

// bf16: a 32-bit word holds elements (2t, 2t+1); fp32: words are the elements themselves.
__device__ __forceinline__ void to_pairs(const uint4& raw, F2 (&z)[4]) {        // 8 bf16
  z[0] = make_f2(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u));
  z[1] = make_f2(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
  z[2] = make_f2(__uint_as_float(raw.z << 16), __uint_as_float(raw.z & 0xFFFF0000u));
  z[3] = make_f2(__uint_as_float(raw.w << 16), __uint_as_float(raw.w & 0xFFFF0000u));
}
__device__ __forceinline__ void to_pairs(const uint4& raw, F2 (&z)[2]) {        // 4 fp32
  z[0] = make_f2(__uint_as_float(raw.x), __uint_as_float(raw.y));
  z[1] = make_f2(__uint_as_float(raw.z), __uint_as_float(raw.w));
}

// out = ReLU(acc * inv + bias), stored in the feature type
__device__ __forceinline__ void finish_row(bf16* dst, const F2 (&acc)[4], float inv, const float (&bs)[8]) {
  uint32_t w[4];
  const F2 i2 = make_f2(inv, inv);
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    F2 o = make_f2(bs[2 * t], bs[2 * t + 1]);
    fma2(o, acc[t], i2);
    float lo, hi;
    split_f2(o, lo, hi);
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(w[t]) : "f"(hi), "f"(lo));   // ReLU inside the rounding
  }
  *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ void finish_row(float* dst, const F2 (&acc)[2], float inv, const float (&bs)[4]) {
  float o[4];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    float lo, hi;
    split_f2(acc[t], lo, hi);
    o[2 * t] = fmaxf(fmaf(lo, inv, bs[2 * t]), 0.f);
    o[2 * t + 1] = fmaxf(fmaf(hi, inv, bs[2 * t + 1]), 0.f);
  }
  *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[1], o[2], o[3]);
}

// out = ReLU(acc * inv + bias) kept in fp32, as register pairs (for the fused per-graph readout)
template <int NP>
__device__ __forceinline__ void finish_row_f32(const F2 (&acc)[NP], float inv, const float (&bs)[2 * NP],
                                               F2 (&o)[NP]) {
  const F2 i2 = make_f2(inv, inv);
#pragma unroll
  for (int t = 0; t < NP; ++t) {
    F2 v = make_f2(bs[2 * t], bs[2 * t + 1]);
    fma2(v, acc[t], i2);
    float lo, hi;
    split_f2(v, lo, hi);
    o[t] = make_f2(fmaxf(lo, 0.f), fmaxf(hi, 0.f));
  }
}

// Rare path of the running softmax: the reference exponent is moved up only when a score exceeds
// it by more than 32 (so every weight stays below 2^32 and nothing overflows); kept a real branch so
// that the common path carries no rescaling arithmetic.
template <int NP>
__device__ __forceinline__ void raise_reference(float ev, float& m, float& l, F2 (&acc)[NP]) {
  asm volatile("" ::: "memory");          // keeps this a real (rarely taken) branch, not predicated code
  const float scale = fast_exp2(m - ev);
  l *= scale;
  const F2 s2 = make_f2(scale, scale);
#pragma unroll
  for (int t = 0; t < NP; ++t) mul2(acc[t], s2);
  m = ev;
}

// One warp's share of a layer.  `next_block()` returns the first row of the warp's next block of up to
// 2^br_shift destination rows, or a negative value when there is none left.  READOUT = true is the last
// attention layer fused with the per-graph sum of Eq. 8: the layer output is not stored; the warp adds
// the rows of its block per graph, in row order, and writes
//   partial[b]           the rows of block b that belong to the graph of the block's first row
//   partial[nblocks + g] the rows of graph g inside the block in which g starts, when that is not at
//                        the block's first row
// (k_global_update_blocks adds them per graph in a fixed order; needs row_begin = win_base = 0, and
// block b = first row >> br_shift).  The ring's barriers are initialised here: call it with no copy of
// this warp in flight.  Returns false when a wait ran out (the caller reports it).
// SEQ: producers taken two at a time are added exactly as if taken singly (one more addition and compare per
// pair); without it the pair's weights are summed first and one overflow test serves both, which is faster
// and equal up to rounding.  Kernels whose results must agree bit for bit use the same setting.
template <typename T, int K, bool READOUT, bool MERGED, int G, int GQ, bool SEQ, typename NextBlock>
__device__ __forceinline__ bool aggregate_warp(
    const CUtensorMap* map_z_p, const CUtensorMap* map_s_p, const int32_t* __restrict__ rowptr,
    const int32_t* __restrict__ col, const T* __restrict__ Z, const float2* __restrict__ scores,
    const float* __restrict__ bias, T* __restrict__ h_out, const Window win,
    const int32_t* __restrict__ seg_id, float* __restrict__ partial, const int32_t nblocks,
    const int32_t* __restrict__ self_idx, const int32_t br_shift, WarpSmem<K, MERGED, G, GQ>& sm,
    NextBlock next_block) {
  const int br = 1 << br_shift;
  constexpr int GV = 4 * GQ;
  constexpr int VEC = VecOf<T>::N;
  constexpr int NP = VEC / 2;
  constexpr int H = 32 * VEC;
  using Smem = WarpSmem<K, MERGED, G, GQ>;
  constexpr uint32_t ZR = Smem::ROW;                  // bytes per gathered row
  constexpr uint32_t SR = MERGED ? ZR : 8 * K;        // distance between consecutive rows' pairs
  constexpr uint32_t GROUP_BYTES = GV * (512 + K * 8);
  constexpr uint32_t ZG = GV * ZR, SG = GV * SR;      // bytes per group in the ring(s)
  constexpr int ZS = int(ZR / sizeof(T));             // elements between rows of the Z buffer (slow path)
  const int lane = threadIdx.x & 31;
  const int c0 = lane * VEC;
  const int head = c0 / (H / K);
  float bs[VEC];
#pragma unroll
  for (int t = 0; t < VEC; ++t) bs[t] = __ldg(bias + c0 + t);
  const uint32_t z_base = smem_u32(&sm.z[0][0][0]);
  const uint32_t s_base = smem_u32(&sm.sc[0][0][0]);
  const uint32_t z_lane = z_base + lane * 16;                // this lane's 16 bytes of slot 0, row 0
  const uint32_t s_lane = MERGED ? z_base + 512 + head * 8   // this lane's head in slot 0, row 0
                                 : s_base + head * 8;
  const uint32_t bar_base = smem_u32(&sm.bar[0]);

  if (lane == 0) {
    for (int g = 0; g < G; ++g) mbar_init(bar_base + 8 * g, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncwarp();

  // ring state, carried across lists: slot and phase parity of the next group to consume
  uint32_t slot = 0, par = 0;
  bool alive = true;

  // lane 0: hand group `gi` of the current list (list rows item[GV gi .. GV gi + GV - 1]) to slot `s`
  auto issue = [&](int gi, uint32_t s) {
    const uint32_t bar = bar_base + 8 * s;
    mbar_expect_tx(bar, GROUP_BYTES);
#pragma unroll
    for (int q = 0; q < GQ; ++q) {
      const int4 it = *reinterpret_cast<const int4*>(&sm.item[gi * GV + q * 4]);
      tma_gather4(z_base + s * ZG + q * 4 * ZR, map_z_p, it.x, it.y, it.z, it.w, bar);
      if (!MERGED) tma_gather4(s_base + s * SG + q * 4 * SR, map_s_p, it.x, it.y, it.z, it.w, bar);
    }
  };

  for (int64_t r0 = next_block(); r0 >= 0 && alive; r0 = next_block()) {
    const int nr = int(min(int64_t(br), win.row_end - r0));
    __syncwarp();
    if (lane < nr) sm.rp[lane] = __ldg(rowptr + r0 + lane);
    if (lane == 0) sm.rp[nr] = __ldg(rowptr + r0 + nr);
    __syncwarp();
    // fused readout: running per-graph sum of this block's rows
    int32_t myseg = 0, cur_g = -1;
    bool first_seg = true;
    F2 rsum[NP];
    if (READOUT) {
      myseg = (lane < nr) ? __ldg(seg_id + r0 + lane) : 0;
#pragma unroll
      for (int t = 0; t < NP; ++t) rsum[t] = make_f2(0.f, 0.f);
    }
    auto flush = [&]() {
      float* dst = partial + size_t(first_seg ? int32_t(r0 >> br_shift) : nblocks + cur_g) * H + c0;
#pragma unroll
      for (int t = 0; t < NP; t += 2) {
        float4 v;
        split_f2(rsum[t], v.x, v.y);
        split_f2(rsum[t + 1], v.z, v.w);
        *reinterpret_cast<float4*>(dst + 2 * t) = v;
      }
    };
    auto add_row = [&](int row_in_block, const F2 (&o)[NP]) {
      const int32_t g = __shfl_sync(0xFFFFFFFFu, myseg, row_in_block);
      if (g != cur_g) {
        if (cur_g >= 0) {
          flush();
          first_seg = false;
#pragma unroll
          for (int t = 0; t < NP; ++t) rsum[t] = make_f2(0.f, 0.f);
        }
        cur_g = g;
      }
#pragma unroll
      for (int t = 0; t < NP; ++t) add2(rsum[t], o[t]);
    };
    int rs = 0;
    while (rs < nr && alive) {
      // as many rows from rs on as keep (rows + producers) within the list
      const int32_t eb = sm.rp[rs];
      const bool fits = (rs + lane < nr) && (lane + 1 + sm.rp[rs + lane + 1] - eb <= ITEMS);
      const uint32_t fmask = __ballot_sync(0xFFFFFFFFu, fits);
      const int cnt = (fmask == 0xFFFFFFFFu) ? 32 : __ffs(~fmask) - 1;
      if (cnt == 0) {
        // a row with more producers than the list holds: plain loads, one producer at a time
        const int32_t lrow = int32_t(r0) + rs - win.win_base;
        const int n = sm.rp[rs + 1] - eb;
        const int32_t srow = self_idx ? __ldg(self_idx + int32_t(r0) + rs) : lrow;
        // pairs of node v: behind its Z row when merged, else in the separate array
        auto pair_of = [&](int32_t v) -> const float2* {
          return MERGED ? reinterpret_cast<const float2*>(Z + size_t(v) * ZS + H) + head
                        : scores + size_t(v) * K + head;
        };
        const float2 self = __ldg(pair_of(srow));
        const float sd = self.y;
        float m = lrelu(self.x + sd), l = 1.f;
        F2 acc[NP];
        to_pairs(__ldg(reinterpret_cast<const uint4*>(Z + size_t(srow) * ZS + c0)), acc);
        for (int t = 0; t < n; ++t) {
          const int32_t j = __ldg(col + eb + t) - win.win_base;
          const float ev = lrelu(__ldg(&pair_of(j)->x) + sd);
          F2 z[NP];
          to_pairs(__ldg(reinterpret_cast<const uint4*>(Z + size_t(j) * ZS + c0)), z);
          if (ev > m + 32.f) raise_reference<NP>(ev, m, l, acc);
          const float p = fast_exp2(ev - m);
          l += p;
          const F2 p2 = make_f2(p, p);
#pragma unroll
          for (int t2 = 0; t2 < NP; ++t2) fma2(acc[t2], p2, z[t2]);
        }
        if (READOUT) {
          F2 o[NP];
          finish_row_f32<NP>(acc, __fdividef(1.f, l), bs, o);
          add_row(rs, o);
        } else {
          finish_row(h_out + size_t(lrow) * H + c0, acc, __fdividef(1.f, l), bs);
        }
        rs += 1;
        continue;
      }
      // ---- the list: for each row its own index, then its producers', all window-relative ----------
      __syncwarp();
      const int total = cnt + (sm.rp[rs + cnt] - eb);
      if (lane < cnt) {
        const int e0 = sm.rp[rs + lane] - eb, n = sm.rp[rs + lane + 1] - eb - e0;
        int pos = lane + e0;
        sm.item[pos++] = self_idx ? __ldg(self_idx + int32_t(r0) + rs + lane)       // where the row's own Z lives
                                  : int32_t(r0) + rs + lane - win.win_base;
        for (int t = 0; t < n; ++t) sm.item[pos++] = __ldg(col + eb + e0 + t) - win.win_base;
      }
      if (lane < GV) sm.item[total + lane] = int32_t(r0) + rs - win.win_base;   // pad the last group
      __syncwarp();
      const int ngroups = (total + GV - 1) / GV;
      if (lane == 0) {
        uint32_t s = slot;
        for (int gi = 0; gi < min(G, ngroups); ++gi) { issue(gi, s); s = (s + 1 == G) ? 0 : s + 1; }
      }

      // ---- consume: rows in order, vectors in list order ----------------------------------------------
      int gi = 0, w = GV;                     // current group of the list, vectors left in it
      uint32_t zp = z_lane + slot * ZG, sp = s_lane + slot * SG;
      if (!wait_all_lanes(bar_base + 8 * slot, par)) alive = false;
      // group finished: refill its slot with group gi + G, move on, wait for the next one
      auto advance = [&]() {
        __syncwarp();
        if (lane == 0 && gi + G < ngroups) issue(gi + G, slot);
        ++gi;
        if (++slot == G) { slot = 0; par ^= 1; }
        zp = z_lane + slot * ZG;
        sp = s_lane + slot * SG;
        w = GV;
        if (gi < ngroups && alive && !wait_all_lanes(bar_base + 8 * slot, par)) alive = false;
      };
      for (int rr = 0; rr < cnt; ++rr) {
        const int n = sm.rp[rs + rr + 1] - sm.rp[rs + rr];
        // the row's own vector opens the running softmax: reference exponent = its score, weight 1
        uint4 raw = lds128(zp);
        float2 sc = lds64(sp);
        zp += ZR; sp += SR;
        if (--w == 0) advance();
        const float sd = sc.y;
        float m = lrelu(sc.x + sd), l = 1.f;
        F2 acc[NP];
        to_pairs(raw, acc);
        int t = 0;
        // two producers at a time while the row and the group at the ring's head both have two left: one
        // pointer step, one ring check and one overflow test for the pair, and two independent chains
        while (n - t >= 2 && w >= 2) {
          const uint4 raw0 = lds128(zp), raw1 = lds128(zp + ZR);
          const float2 sc0 = lds64(sp), sc1 = lds64(sp + SR);
          zp += 2 * ZR; sp += 2 * SR;
          t += 2;
          if ((w -= 2) == 0) advance();
          const float ev0 = lrelu(sc0.x + sd), ev1 = lrelu(sc1.x + sd);
          float p0, p1;
          if (SEQ) {
            // the arithmetic of taking the two one after the other, so that a row's result does not depend on how
            // its producers fall into pairs, i.e. on the ring's geometry
            if (fmaxf(ev0, ev1) > m + 32.f) {
              F2 z[NP];
              if (ev0 > m + 32.f) raise_reference<NP>(ev0, m, l, acc);
              const float pa = fast_exp2(ev0 - m);
              l += pa;
              to_pairs(raw0, z);
              const F2 qa = make_f2(pa, pa);
#pragma unroll
              for (int t2 = 0; t2 < NP; ++t2) fma2(acc[t2], qa, z[t2]);
              if (ev1 > m + 32.f) raise_reference<NP>(ev1, m, l, acc);
              const float pb = fast_exp2(ev1 - m);
              l += pb;
              to_pairs(raw1, z);
              const F2 qb = make_f2(pb, pb);
#pragma unroll
              for (int t2 = 0; t2 < NP; ++t2) fma2(acc[t2], qb, z[t2]);
              continue;
            }
            p0 = fast_exp2(ev0 - m);
            p1 = fast_exp2(ev1 - m);
            l += p0;
            l += p1;
          } else {
            const float evm = fmaxf(ev0, ev1);
            if (evm > m + 32.f) raise_reference<NP>(evm, m, l, acc);
            p0 = fast_exp2(ev0 - m);
            p1 = fast_exp2(ev1 - m);
            l += p0 + p1;
          }
          F2 z0[NP], z1[NP];
          to_pairs(raw0, z0);
          to_pairs(raw1, z1);
          const F2 q0 = make_f2(p0, p0), q1 = make_f2(p1, p1);
#pragma unroll
          for (int t2 = 0; t2 < NP; ++t2) fma2(acc[t2], q0, z0[t2]);
#pragma unroll
          for (int t2 = 0; t2 < NP; ++t2) fma2(acc[t2], q1, z1[t2]);
        }
        for (; t < n; ++t) {
          raw = lds128(zp);
          sc = lds64(sp);
          zp += ZR; sp += SR;
          if (--w == 0) advance();
          const float ev = lrelu(sc.x + sd);
          if (ev > m + 32.f) raise_reference<NP>(ev, m, l, acc);
          const float p = fast_exp2(ev - m);
          l += p;
          F2 z[NP];
          to_pairs(raw, z);
          const F2 p2 = make_f2(p, p);
#pragma unroll
          for (int t2 = 0; t2 < NP; ++t2) fma2(acc[t2], p2, z[t2]);
        }
        if (READOUT) {
          F2 o[NP];
          finish_row_f32<NP>(acc, __fdividef(1.f, l), bs, o);
          add_row(rs + rr, o);
        } else {
          finish_row(h_out + size_t(int32_t(r0) + rs + rr - win.win_base) * H + c0, acc, __fdividef(1.f, l), bs);
        }
      }
      if (w != GV) {                           // the list ended inside a group: retire it without waiting
        __syncwarp();
        if (++slot == G) { slot = 0; par ^= 1; }
      }
      rs += cnt;
    }
    if (READOUT && cur_g >= 0) flush();
  }
  return alive;
}

// ---- host side ----------------------------------------------------------------------------------
// Z rows followed by their half-score pairs, as rows of 32-bit words; gather4 takes boxes one row high.
inline bool make_merged_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint32_t row_bytes) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {row_bytes / 4, rows};      // rows of 32-bit words: features, then the pairs
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {row_bytes / 4, 1};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace aggtma
}  // namespace xrl

// Node-update layer (paper Eq. 6) on the tensor cores for bf16 storage:
//   h0_i = ReLU(W0^T [ sum_{j->i} shape_j | onehot(op_i) | shape_i ] + b0)
// written as one dense product X . W0ext with fp32 accumulation in tensor memory.  The rows of X
// are built on the fly by gather threads, one node per thread, as 16-byte pieces of 8 bf16:
//   piece 0        bf16(ebar)            ebar = fp32 sum of the producers' shape features
//   piece 1        the node's own shape features (already bf16)
//   pieces 2..     the one-hot operator id
//   next piece     bf16(ebar - bf16(ebar)): with it the product sees ebar to ~2^-17 relative
//   next piece     (1, 1, 0, ...) against two rows holding b0 split the same way into high and low
//                  bf16 parts, so that the bias enters with fp32-like accuracy
// W0ext^T (K-major, built once when the weights are set) stays resident in shared memory; three
// gather groups of 128 threads fill three A stages in turn; one thread issues tcgen05.mma; four
// epilogue warps apply the ReLU, round to bf16 and store the tile with TMA.  The layer writes H b
// bytes per node and reads ~30: it is bound by the HBM write stream.
//
// All waits are bounded; a timeout raises XRL_ERR_TIMEOUT in the status word and the kernel
// frees its tensor memory and returns.
#include "xrl_umma.cuh"

namespace xrl {

using namespace umma;

namespace {

constexpr int BM = 128;
constexpr int CHUNK_BYTES = BM * 128;        // 128 rows x 64 bf16, 128-byte swizzled
constexpr int A_STAGE_BYTES = 2 * CHUNK_BYTES;
constexpr int GROUPS = 3;                    // gather groups = A stages
constexpr int kThreads = 32 * (1 + 4 + 4 * GROUPS);   // warp 0 MMA, 1..4 epilogue, 5.. gather

template <int H> struct ECfg {
  static constexpr int B_BYTES = 2 * H * 128;            // two K chunks of N = H rows
  static constexpr int OFF_A = B_BYTES;
  static constexpr int OFF_OUT = OFF_A + GROUPS * A_STAGE_BYTES;
  static constexpr int OFF_BAR = OFF_OUT + 2 * CHUNK_BYTES;
  static constexpr int NUM_BARS = 1 + 2 * GROUPS + 4;
  static constexpr int OFF_TMEM = OFF_BAR + NUM_BARS * 8;
  static constexpr int SMEM_BYTES = OFF_TMEM + 16;
  static constexpr int TMEM_COLS = 2 * H;
};

template <int H>
__global__ void __launch_bounds__(kThreads, 1)
k_embed_umma(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_h,
             const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
             const int32_t* __restrict__ op, const bf16* __restrict__ shape,
             const int32_t* __restrict__ row_list, int row_begin, int rows, int op_pieces, int ksteps,
             int32_t* status, const bf16* __restrict__ eattr) {
  using C = ECfg<H>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t base = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = (rows + BM - 1) / BM;
  const int kchunks = (ksteps + 3) / 4;

  if ((base & 1023u) != 0) {
    if (threadIdx.x == 0) raise(status, XRL_ERR_UNSUPPORTED);
    return;
  }
  const uint32_t bar0 = base + C::OFF_BAR;
  const uint32_t bar_w = bar0;
  auto bar_a_full = [&](int s) { return bar0 + 8u * (1 + s); };
  auto bar_a_empty = [&](int s) { return bar0 + 8u * (1 + GROUPS + s); };
  auto bar_acc_full = [&](int b) { return bar0 + 8u * (1 + 2 * GROUPS + b); };
  auto bar_acc_empty = [&](int b) { return bar0 + 8u * (1 + 2 * GROUPS + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_TMEM);

  if (threadIdx.x == 0) {
    tmem_slot[1] = 0;
    mbar_init(bar_w, 1);
    for (int s = 0; s < GROUPS; ++s) { mbar_init(bar_a_full(s), 128); mbar_init(bar_a_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_acc_full(b), 1); mbar_init(bar_acc_empty(b), 128); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(uint32_t(C::TMEM_COLS)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---- weights in, then MMA issue ----------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(H >> 3) << 17) |
                                 (uint32_t(BM >> 4) << 24);
      mbar_expect_tx(bar_w, uint32_t(kchunks) * H * 128);
      for (int kc = 0; kc < kchunks; ++kc) tma_load_2d(base + kc * H * 128, &map_w, kc * KCH, 0, bar_w);
      bool ok = mbar_wait(bar_w, 0);
      tc_fence_after();
      uint32_t lt = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
        const int buf = lt & 1, s = lt % GROUPS;
        const uint32_t use = lt >> 1;
        if (use > 0 && !mbar_wait(bar_acc_empty(buf), (use - 1) & 1)) { ok = false; break; }
        if (!mbar_wait(bar_a_full(s), (lt / GROUPS) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + uint32_t(buf * H);
        const uint32_t a_addr = base + C::OFF_A + s * A_STAGE_BYTES;
        for (int ks = 0; ks < ksteps; ++ks)
          tc_mma(tmem_d, smem_desc(a_addr + (ks >> 2) * CHUNK_BYTES + (ks & 3) * 32),
                 smem_desc(base + (ks >> 2) * H * 128 + (ks & 3) * 32), idesc, ks != 0 ? 1u : 0u);
        tc_commit(bar_a_empty(s));
        tc_commit(bar_acc_full(buf));
      }
      if (!ok) raise(status, XRL_ERR_TIMEOUT);
    }
  } else if (warp <= 4) {
    // ---- epilogue: ReLU, round to bf16, TMA store ---------------------------------------------------
    const int q = warp & 3;
    const int row_in_tile = q * 32 + lane;
    const bool leader = (threadIdx.x == 32);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint32_t lt = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++lt) {
      const int buf = lt & 1;
      uint32_t okw = 1;
      if (lane == 0) okw = mbar_wait(bar_acc_full(buf), (lt >> 1) & 1) ? 1u : 0u;
      okw = __shfl_sync(0xFFFFFFFFu, okw, 0);
      if (!okw && lane == 0) { *abort_flag = 1; raise(status, XRL_ERR_TIMEOUT); }
      epi_barrier();
      if (*abort_flag) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(q * 32) << 16) + uint32_t(buf * H);
      for (int c = 0; c < H / 64; ++c) {
        uint32_t v[2][32];
        tc_ld32(taddr + c * 64, v[0]);
        tc_ld32(taddr + c * 64 + 32, v[1]);
        tc_wait_ld();
        if (leader) tma_wait_read<1>();
        epi_barrier();
        uint8_t* stage = smem + C::OFF_OUT + (c & 1) * CHUNK_BYTES + row_in_tile * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t* z = &v[j >> 2][(j & 3) * 8];
          uint4 pk;
          pk.x = pack_bf16x2(fmaxf(__uint_as_float(z[0]), 0.f), fmaxf(__uint_as_float(z[1]), 0.f));
          pk.y = pack_bf16x2(fmaxf(__uint_as_float(z[2]), 0.f), fmaxf(__uint_as_float(z[3]), 0.f));
          pk.z = pack_bf16x2(fmaxf(__uint_as_float(z[4]), 0.f), fmaxf(__uint_as_float(z[5]), 0.f));
          pk.w = pack_bf16x2(fmaxf(__uint_as_float(z[6]), 0.f), fmaxf(__uint_as_float(z[7]), 0.f));
          *reinterpret_cast<uint4*>(stage + ((j ^ (row_in_tile & 7)) << 4)) = pk;
        }
        fence_async_smem();
        epi_barrier();
        if (leader) {
          tma_store_2d(&map_h, base + C::OFF_OUT + (c & 1) * CHUNK_BYTES, c * 64, tile * BM);
          tma_commit();
        }
      }
      tc_fence_before();
      mbar_arrive(bar_acc_empty(buf));
    }
    if (leader) tma_wait_all();
  } else {
    // ---- gather: one node per thread, group g fills stage g for its share of the tiles -------------
    const int g = (warp - 5) >> 2;
    const int r = ((warp - 5) & 3) * 32 + lane;               // row inside the tile
    const int pieces = 2 * ksteps;                            // 16-byte pieces per row actually read
    uint32_t lt = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++lt) {
      if (int(lt % GROUPS) != g) continue;
      const int lrow = tile * BM + r;
      float e[kS];
#pragma unroll
      for (int s = 0; s < kS; ++s) e[s] = 0.f;
      uint4 own = make_uint4(0, 0, 0, 0);
      int o = -1;
      if (lrow < rows) {
        const int32_t row = row_list ? __ldg(row_list + lrow) : row_begin + lrow;   // listed rows are written densely
        const int32_t e0 = __ldg(rowptr + row), e1 = __ldg(rowptr + row + 1);
        own = __ldg(reinterpret_cast<const uint4*>(shape + size_t(row) * kS));
        o = __ldg(op + row);
        for (int32_t ed = e0; ed < e1; ++ed) {
          float f[kS];
          // the producer's shape features, or the edge's own attributes (kept in slot order)
          const bf16* src = eattr ? eattr + size_t(ed) * kS : shape + size_t(__ldg(col + ed)) * kS;
          unpack(__ldg(reinterpret_cast<const uint4*>(src)), f);
#pragma unroll
          for (int s = 0; s < kS; ++s) e[s] += f[s];
        }
      }
      float hi[kS], lo[kS];
#pragma unroll
      for (int s = 0; s < kS; ++s) {
        hi[s] = __bfloat162float(__float2bfloat16_rn(e[s]));
        lo[s] = e[s] - hi[s];
      }
      const uint32_t use = lt / GROUPS;
      if (use > 0 && !mbar_wait(bar_a_empty(g), (use - 1) & 1)) { raise(status, XRL_ERR_TIMEOUT); break; }
      uint8_t* arow = smem + C::OFF_A + g * A_STAGE_BYTES + r * 128;
      for (int pc = 0; pc < pieces; ++pc) {
        uint4 val = make_uint4(0, 0, 0, 0);
        if (pc == 0) val = pack(hi);
        else if (pc == 1) val = own;
        else if (pc < 2 + op_pieces) {
          if (o >= 0 && (o >> 3) == pc - 2) {                 // bf16 1.0 = 0x3F80 at element o % 8
            const uint32_t one = 0x3F80u << (16 * (o & 1));
            const int w = (o & 7) >> 1;
            val.x = w == 0 ? one : 0u; val.y = w == 1 ? one : 0u;
            val.z = w == 2 ? one : 0u; val.w = w == 3 ? one : 0u;
          }
        } else if (pc == 2 + op_pieces) val = pack(lo);
        else if (pc == 3 + op_pieces) val.x = (lrow < rows) ? 0x3F803F80u : 0u;
        *reinterpret_cast<uint4*>(arow + (pc >> 3) * CHUNK_BYTES + (((pc & 7) ^ (r & 7)) << 4)) = val;
      }
      fence_async_smem();
      mbar_arrive(bar_a_full(g));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"(uint32_t(C::TMEM_COLS)) : "memory");
  }
}

// W0ext^T [H x kpad] bf16, K-major: column k of node-update input piece layout (see the header).
__global__ void k_build_w0ext(const bf16* __restrict__ W0, const float* __restrict__ b0,
                              bf16* __restrict__ out, int H, int T, int op_pieces, int kpad) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= H * kpad) return;
  const int n = i / kpad, k = i - n * kpad;
  const int k_lo = 16 + 8 * op_pieces, k_b = k_lo + 8;
  float v = 0.f;
  if (k < 8) v = __bfloat162float(W0[size_t(k) * H + n]);                          // edge aggregate (high)
  else if (k < 16) v = __bfloat162float(W0[size_t(kS + T + (k - 8)) * H + n]);     // own shape
  else if (k < 16 + T) v = __bfloat162float(W0[size_t(kS + (k - 16)) * H + n]);    // one-hot operator
  else if (k >= k_lo && k < k_lo + 8) v = __bfloat162float(W0[size_t(k - k_lo) * H + n]);  // aggregate (low)
  else if (k == k_b) v = __bfloat162float(__float2bfloat16_rn(b0[n]));
  else if (k == k_b + 1) v = b0[n] - __bfloat162float(__float2bfloat16_rn(b0[n]));
  out[i] = __float2bfloat16_rn(v);
}

template <int H>
int launch_h(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op,
             const void* shape, const void* w0ext_t, void* h, Window win, const int32_t* row_list,
             int32_t* status, cudaStream_t st, const void* eattr) {
  using C = ECfg<H>;
  static bool attr_set[64] = {};
  if (!ensure_dynamic_smem(k_embed_umma<H>, C::SMEM_BYTES, attr_set)) return -1;
  const int op_pieces = (d.T + 7) / 8;
  const int ksteps = (4 + op_pieces + 1) / 2;
  const int kpad = ((ksteps + 3) / 4) * KCH;
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  bf16* hp = static_cast<bf16*>(h) + size_t(win.row_begin - win.win_base) * H;
  CUtensorMap mw, mh;
  if (!make_map(&mw, w0ext_t, H, uint64_t(kpad), H) || !make_map(&mh, hp, uint64_t(rows), H, BM)) return -1;
  const int tiles = int((rows + BM - 1) / BM);
  const int grid = tiles < kNumSMs ? tiles : kNumSMs;
  k_embed_umma<H><<<grid, kThreads, C::SMEM_BYTES, st>>>(mw, mh, rowptr, col, op,
                                                         static_cast<const bf16*>(shape), row_list,
                                                         win.row_begin, int(rows), op_pieces, ksteps, status,
                                                         static_cast<const bf16*>(eattr));
  return 1;
}

}  // namespace

bool embed_umma_supported(const Dims& d) {
  return d.dtype == XRL_BF16 && (d.H == 128 || d.H == 256) && d.T <= 96 && encode_fn() != nullptr;
}

// Elements in one row of W0ext^T (a multiple of 64).
int embed_umma_kpad(const Dims& d) {
  const int op_pieces = (d.T + 7) / 8;
  return (((4 + op_pieces + 1) / 2 + 3) / 4) * KCH;
}

void build_w0ext(const Dims& d, const void* W0_store, const float* b0, void* out, cudaStream_t st) {
  const int kpad = embed_umma_kpad(d), n = d.H * kpad;
  k_build_w0ext<<<(n + 255) / 256, 256, 0, st>>>(static_cast<const bf16*>(W0_store), b0,
                                                  static_cast<bf16*>(out), d.H, d.T, (d.T + 7) / 8, kpad);
}

int launch_embed_umma(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op,
                      const void* shape, const void* w0ext_t, void* h, Window win, int32_t* status,
                      cudaStream_t st, const int32_t* row_list, const void* eattr) {
  if (int64_t(win.row_end) - win.row_begin <= 0) return 0;
  if (d.H == 256) return launch_h<256>(d, rowptr, col, op, shape, w0ext_t, h, win, row_list, status, st, eattr);
  return launch_h<128>(d, rowptr, col, op, shape, w0ext_t, h, win, row_list, status, st, eattr);
}

}  // namespace xrl

// All attention layers of a small step in one cooperative launch (paper Section 3.4: k graph-attention
// layers back to back, Eq. 7), for bf16 storage and hidden 256.
//
// A step of the paper's size (tens of candidates, ten to twenty thousand nodes) is a handful of 128-row
// tiles per SM at most; launched layer by layer it is bound by the fill and drain of 2 L small kernels.
// Here one persistent CTA per SM owns the tiles t = blockIdx.x, blockIdx.x + gridDim.x, ... for the
// whole stack and alternates between two phases per layer:
//   transform   Z = h W (+ half-scores) of its tiles: TMA producer, tcgen05 issuer and four epilogue
//               warps, exactly the roles of the one-layer kernel;
//   attention   score / softmax / aggregate of the rows of the same tiles: every warp takes blocks of
//               destination rows and gathers the producers' Z rows with the TMA unit.
// The attention phase reads Z rows of other CTAs' tiles, so a grid-wide barrier separates it from the
// transform phase (the launch is cooperative, so all CTAs are resident; the barrier is a counter in
// global memory that every CTA adds to and then polls, with a limit like every other wait); the next
// transform reads only rows this CTA has just written, so a CTA barrier is enough there.  Z alternates between two buffers: a CTA that is already
// transforming layer l + 1 must not overwrite rows a slower CTA still gathers for layer l.  W of the
// next layer streams into shared memory during the attention phase, whose gather rings live where the
// transform's A stages and output staging are.  Tensor memory is allocated once.
//
// Arithmetic, summation order and (for the last layer fused with the Eq. 8 sum) the layout of the
// partial sums are those of the one-layer kernels: the results are bit-identical.
//
// Every mbarrier wait is bounded; a CTA whose wait ran out raises XRL_ERR_TIMEOUT, skips the work of
// the remaining phases and still arrives at every grid barrier.
#include "xrl_agg_tma.cuh"
#include "xrl_xform_umma.cuh"

namespace xrl {

using namespace umma;

namespace {

constexpr int H = 256;
constexpr int kWarps = 16;             // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue; all 16 in the attention phase
constexpr int kThreads = 32 * kWarps;
#ifndef XRL_COOP_RING_GROUPS
#define XRL_COOP_RING_GROUPS 2
#endif
#ifndef XRL_COOP_RING_GATHERS
#define XRL_COOP_RING_GATHERS 1
#endif
#ifndef XRL_COOP_ATT_WARPS
#define XRL_COOP_ATT_WARPS 16
#endif
constexpr int AG = XRL_COOP_RING_GROUPS, AGQ = XRL_COOP_RING_GATHERS;   // per warp: AG gather groups of 4 AGQ rows in flight
constexpr int kAttWarps = XRL_COOP_ATT_WARPS;                             // warps that take part in the attention phase
constexpr int kMaxLayers = 8;
using XC = xform::Cfg<H>;

struct CoopParams {
  CUtensorMap map_h;                   // node features [rows x H] bf16: A tiles of the transform
  CUtensorMap map_zs[2];               // the two Z buffers as [rows x H] bf16 with the merged row stride: stores
  CUtensorMap map_zg[2];               // the same buffers as merged rows of 32-bit words: gathers
  CUtensorMap map_w[kMaxLayers];       // W^T of each layer
  const float* a_src[kMaxLayers];
  const float* a_dst[kMaxLayers];
  const float* bias[kMaxLayers];
  bf16* Z[2];
  bf16* h;
  const int32_t* rowptr;
  const int32_t* col;
  const int32_t* seg_id;
  float* partial;                      // non-null: the last layer leaves per-block sums instead of node features
  int32_t* status;
  uint32_t* sync;                      // [0] arrivals at the grid barriers of this launch, [1] CTAs that have finished
  int32_t rows, layers, K, nblocks, br_shift, z_row_bytes;
};

// Grid-wide barrier number `k` (1, 2, ...) of a launch of `ctas` resident CTAs: called by every thread.  Plain
// stores before it are visible to every CTA after it.  False when the others did not arrive within the time
// limit (the caller reports it and carries on: it still arrives at the later barriers).  ok_word: a word of shared
// memory for the outcome.
__device__ __forceinline__ bool grid_barrier(uint32_t* counter, uint32_t k, uint32_t ctas, volatile uint32_t* ok_word) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(counter, 1u);
    const uint32_t target = k * ctas;
    volatile uint32_t* c = counter;
    // a poll is a round trip to L2 (a good half microsecond): 2^21 of them are about a second
    uint32_t ok = 0;
    for (int it = 0; it < (1 << 21); ++it)
      if (*c >= target) { ok = 1; break; }
    __threadfence();
    *ok_word = ok;
  }
  __syncthreads();
  return *ok_word != 0;
}

template <int K>
__global__ void __launch_bounds__(kThreads, 1) k_layers_coop(const __grid_constant__ CoopParams p) {
  using Ring = aggtma::WarpSmem<K, true, AG, AGQ>;
  static_assert(sizeof(Ring) * kAttWarps <= size_t(XC::OFF_AVEC - XC::OFF_A), "gather rings must fit behind W");
  static_assert(kAttWarps <= kWarps, "attention warps are warps of the CTA");
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t base = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = (p.rows + xform::BM - 1) / xform::BM;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + XC::OFF_TMEM);
  // [1] is set by the epilogue warps between their own barriers (they read it there), [2] by every other role,
  // [3] holds the outcome of the last grid barrier
  volatile uint32_t* abort_role = tmem_slot + 2;
  auto aborted = [&]() { return (abort_role[-1] | abort_role[0]) != 0; };    // read between CTA barriers only
  float* avec = reinterpret_cast<float*>(smem + XC::OFF_AVEC);

  if (threadIdx.x == 0) {
    // the swizzled tiles need 1024-byte alignment (the same in every CTA)
    tmem_slot[1] = 0;
    tmem_slot[2] = (base & 1023u) != 0 ? 1u : 0u;
    if (tmem_slot[2]) raise(p.status, XRL_ERR_UNSUPPORTED);
    xform::init_barriers<H>(base);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_slot)), "r"(uint32_t(XC::TMEM_COLS)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  uint32_t prod_it = 0, mma_it = 0, mma_lt = 0, epi_lt = 0;     // ring / accumulator positions, kept across layers
  if (threadIdx.x == 0 && !aborted()) xform::load_w<H>(base, &p.map_w[0]);

  const int my_tiles = (num_tiles - int(blockIdx.x) + int(gridDim.x) - 1) / int(gridDim.x);
  const int blk_bits = 7 - p.br_shift;                           // blocks per 128-row tile = 2^blk_bits
  const Window win{0, p.rows, 0};

  for (int l = 0; l < p.layers; ++l) {
    const int zb = l & 1;
    // attention vectors pre-multiplied by log2(e): the half-scores are consumed by an exp2 softmax
    for (int t = threadIdx.x; t < H; t += kThreads) {
      avec[t] = __ldg(p.a_src[l] + t) * kLog2e;
      avec[H + t] = __ldg(p.a_dst[l] + t) * kLog2e;
    }
    __syncthreads();

    // ---- transform phase: Z[zb] rows (and their half-score pairs) of this CTA's tiles --------------------
    if (!aborted()) {
      if (warp == 0) {
        if (lane == 0 && !xform::produce_tiles<H>(base, &p.map_h, blockIdx.x, gridDim.x, num_tiles, prod_it)) {
          raise(p.status, XRL_ERR_TIMEOUT);
          xform::drain_producer<H>(base, prod_it, uint32_t(l & 1));
          *abort_role = 1;
        }
      } else if (warp == 1) {
        if (lane == 0 && !xform::mma_tiles<H>(base, tmem_base, blockIdx.x, gridDim.x, num_tiles, mma_it, mma_lt,
                                              uint32_t(l & 1))) {
          raise(p.status, XRL_ERR_TIMEOUT);
          *abort_role = 1;
        }
      } else if (warp < 6) {
        float2* pairs = reinterpret_cast<float2*>(reinterpret_cast<char*>(p.Z[zb]) + size_t(H) * 2);
        xform::epilogue_tiles<H>(smem, base, tmem_base, &p.map_zs[zb], pairs, p.z_row_bytes / 8, p.rows, K,
                                 blockIdx.x, gridDim.x, num_tiles, epi_lt, threadIdx.x == 64, p.status);
      }
    }
    // the pairs were written with plain stores and are gathered by other CTAs' TMA units
    fence_async_all();
    tc_fence_before();
    if (!grid_barrier(p.sync, uint32_t(l + 1), gridDim.x, tmem_slot + 3) && threadIdx.x == 0) {
      raise(p.status, XRL_ERR_TIMEOUT);
      *abort_role = 1;
    }
    fence_async_all();
    __syncthreads();
    // every accumulator of the transform phase has been read, so all its MMAs have completed: W may be replaced.
    // (Issued only now: a thread's proxy fence waits for the copies it has in flight.)
    if (threadIdx.x == 0 && l + 1 < p.layers && !aborted()) xform::load_w<H>(base, &p.map_w[l + 1]);

    // ---- attention phase: rows of the same tiles; the rings take the place of the A stages and staging ---
    if (!aborted() && warp < kAttWarps) {
      Ring& sm = reinterpret_cast<Ring*>(smem + XC::OFF_A)[warp];
      const int total_blocks = my_tiles << blk_bits;
      int j = warp;
      auto next_block = [&]() -> int64_t {
        while (j < total_blocks) {
          const int k = j >> blk_bits, blk = j & ((1 << blk_bits) - 1);
          j += kAttWarps;
          const int64_t r0 = (int64_t(blockIdx.x) + int64_t(k) * gridDim.x) * xform::BM + (int64_t(blk) << p.br_shift);
          if (r0 < p.rows) return r0;
        }
        return int64_t(-1);
      };
      bool alive;
      if (p.partial != nullptr && l == p.layers - 1)
        alive = aggtma::aggregate_warp<bf16, K, true, true, AG, AGQ, true>(
            &p.map_zg[zb], &p.map_zg[zb], p.rowptr, p.col, p.Z[zb], nullptr, p.bias[l], p.h, win, p.seg_id,
            p.partial, p.nblocks, nullptr, p.br_shift, sm, next_block);
      else
        alive = aggtma::aggregate_warp<bf16, K, false, true, AG, AGQ, true>(
            &p.map_zg[zb], &p.map_zg[zb], p.rowptr, p.col, p.Z[zb], nullptr, p.bias[l], p.h, win, p.seg_id,
            nullptr, p.nblocks, nullptr, p.br_shift, sm, next_block);
      if (!alive) {
        if (lane == 0) { raise(p.status, XRL_ERR_TIMEOUT); *abort_role = 1; }
        for (int t = 0; t < 100; ++t) __nanosleep(10000);     // give copies still in flight time to land
      }
      // the ring's barriers lie where the next transform phase loads its tiles
      __syncwarp();
      if (lane == 0)
        for (int g = 0; g < AG; ++g)
          asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&sm.bar[g])) : "memory");
    }
    // the rows of h this CTA has written with plain stores are loaded by its own TMA unit next
    fence_async_all();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_base), "r"(uint32_t(XC::TMEM_COLS)) : "memory");
  }
  // the last CTA to finish leaves the counters at zero for the next launch (every CTA has left the last barrier
  // before it counts itself as finished)
  if (threadIdx.x == 0 && atomicAdd(p.sync + 1, 1u) == gridDim.x - 1) {
    p.sync[0] = 0;
    p.sync[1] = 0;
    __threadfence();
  }
}

template <int K>
int launch_k(const CoopParams& p, int grid, cudaStream_t st) {
  static bool attr_set[64] = {};
  if (!ensure_dynamic_smem(k_layers_coop<K>, XC::SMEM_BYTES, attr_set)) return -1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = XC::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, k_layers_coop<K>, p) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return 1;
}

}  // namespace

// Row counts this kernel is meant for: at most a few tiles per SM.
constexpr int64_t kCoopMaxRows = 65536;
int64_t layers_coop_max_rows() { return kCoopMaxRows; }

bool layers_coop_supported(const Dims& d, int layers, int64_t rows) {
  return d.dtype == XRL_BF16 && d.H == H && d.zmerged && (d.K == 4 || d.K == 8) && layers >= 1 &&
         layers <= kMaxLayers && rows > 0 && rows <= kCoopMaxRows && encode_fn() != nullptr;
}

// Layers 0 .. layers - 1 of the attention stack over rows [0, rows): reads and overwrites h; Z0 / Z1 are two
// buffers of `rows` merged Z rows.  With `partial` the last layer leaves the per-block sums of Eq. 8 there
// (blocks of 2^aggregate_block_shift(rows) rows, as the one-layer kernel does) and does not write h.
// `sync`: two zeroed 32-bit words of device memory that only launches of this kernel on one stream touch.
// Returns kernels launched, or -1 when the shape is not handled or the launch was refused.
int launch_layers_coop(const Dims& d, const DevWeights& dw, int layers, void* h, void* Z0, void* Z1,
                       const int32_t* rowptr, const int32_t* col, int64_t rows, const int32_t* seg_id,
                       float* partial, int32_t* status, uint32_t* sync, cudaStream_t st) {
  if (!layers_coop_supported(d, layers, rows) || sync == nullptr) return -1;
  CoopParams p;
  const size_t zrow = z_row_bytes(d);
  void* Zs[2] = {Z0, Z1};
  if (!make_map(&p.map_h, h, uint64_t(rows), H, xform::BM)) return -1;
  for (int i = 0; i < 2; ++i) {
    if (!make_map(&p.map_zs[i], Zs[i], uint64_t(rows), H, xform::BM, zrow) ||
        !aggtma::make_merged_map(&p.map_zg[i], Zs[i], uint64_t(rows), uint32_t(zrow)))
      return -1;
    p.Z[i] = static_cast<bf16*>(Zs[i]);
  }
  for (int l = 0; l < kMaxLayers; ++l) {
    const LayerWeights& lw = dw.layer[l < layers ? l : 0];
    if (!make_map(&p.map_w[l], lw.Wt, H, H, H)) return -1;
    p.a_src[l] = lw.a_src; p.a_dst[l] = lw.a_dst; p.bias[l] = lw.b;
  }
  p.h = static_cast<bf16*>(h);
  p.rowptr = rowptr; p.col = col; p.seg_id = seg_id; p.partial = partial; p.status = status; p.sync = sync;
  p.rows = int32_t(rows); p.layers = layers; p.K = d.K;
  p.br_shift = aggregate_block_shift(rows);
  p.nblocks = int32_t((rows + (int64_t(1) << p.br_shift) - 1) >> p.br_shift);
  p.z_row_bytes = int32_t(zrow);
  const int tiles = int((rows + xform::BM - 1) / xform::BM);
  const int grid = tiles < kNumSMs ? tiles : kNumSMs;
  switch (d.K) {
    case 4: return launch_k<4>(p, grid, st);
    case 8: return launch_k<8>(p, grid, st);
    default: return -1;
  }
}

}  // namespace xrl

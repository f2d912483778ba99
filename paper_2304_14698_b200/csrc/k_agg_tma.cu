// Edge score / segment softmax / weighted aggregate of a graph-attention layer (paper Eq. 7) for
// 512-byte feature rows (hidden 256 in bf16, 128 in fp32), with the gathers done by the TMA engine.
//
// A warp takes a block of up to 32 consecutive destination rows and lists the rows of Z it needs
// (each destination's own row, then its producers').  One lane hands the list to the TMA unit four
// rows at a time (cp.async.bulk.tensor ... tile::gather4, one instruction per four 512-byte rows,
// a second one for the four rows of half-score pairs); the data lands in a small per-warp ring in
// shared memory and completion is signalled on an mbarrier.  The 32 lanes then only read their
// 16 bytes of each row from shared memory and do the arithmetic: LeakyReLU score, running-maximum
// softmax with exp2 (the half-scores are stored multiplied by log2 e), fp32 accumulation, bias,
// ReLU.  No lane spends instructions on gather addresses.
//
// Every wait is bounded; on expiry the warp records XRL_ERR_TIMEOUT and stops.
#include "xrl_agg_tma.cuh"

namespace xrl {

using namespace umma;
using namespace aggtma;

namespace {

constexpr int TW = 4;            // warps per CTA
#ifndef XRL_AGG_GROUPS
#define XRL_AGG_GROUPS 2
#endif
#ifndef XRL_AGG_CTAS
#define XRL_AGG_CTAS 5
#endif
#ifndef XRL_AGG_GATHERS
#define XRL_AGG_GATHERS 2
#endif
constexpr int G = XRL_AGG_GROUPS;   // gather groups in flight per warp
constexpr int GQ = XRL_AGG_GATHERS; // gathers (of four rows each) per group: one barrier, one wait per group

// One layer per launch: warp w of the grid takes blocks w, w + (warps of the grid), ... of 2^br_shift
// destination rows (32 in large launches; small ones take 16 or 8, see aggregate_block_shift: with few
// rows a 32-row block per warp leaves most warps idle).  SEQ: see aggregate_warp; set for the small launches that
// the all-layers kernel can replace, whose results it must reproduce bit for bit.
template <typename T, int K, bool READOUT, bool MERGED, bool SEQ>
__global__ void __launch_bounds__(TW * 32, XRL_AGG_CTAS)
k_aggregate_tma(const __grid_constant__ CUtensorMap map_z, const __grid_constant__ CUtensorMap map_s,
                const int32_t* __restrict__ rowptr, const int32_t* __restrict__ col,
                const T* __restrict__ Z, const float2* __restrict__ scores,
                const float* __restrict__ bias, T* __restrict__ h_out, Window win,
                const int32_t* __restrict__ seg_id, float* __restrict__ partial, int32_t nblocks,
                const int32_t* __restrict__ self_idx, int32_t* status, int32_t br_shift) {
  using Smem = WarpSmem<K, MERGED, G, GQ>;
  extern __shared__ __align__(128) uint8_t tma_smem_raw[];
  Smem& sm = reinterpret_cast<Smem*>(tma_smem_raw)[threadIdx.x >> 5];
  const int64_t step = int64_t((gridDim.x * blockDim.x) >> 5) << br_shift;
  int64_t next = int64_t(win.row_begin) + (int64_t((blockIdx.x * blockDim.x + threadIdx.x) >> 5) << br_shift);
  const bool alive = aggregate_warp<T, K, READOUT, MERGED, G, GQ, SEQ>(
      &map_z, &map_s, rowptr, col, Z, scores, bias, h_out, win, seg_id, partial, nblocks, self_idx, br_shift, sm,
      [&]() -> int64_t {
        const int64_t r = next;
        next += step;
        return r < win.row_end ? r : int64_t(-1);
      });
  if (!alive) {
    if ((threadIdx.x & 31) == 0) raise(status, XRL_ERR_TIMEOUT);
    for (int t = 0; t < 100; ++t) __nanosleep(10000);     // give copies still in flight time to land
  }
}

}  // namespace

// log2 of the destination rows one warp takes per block: 32, or 16 / 8 when 32-row blocks would not give every
// resident warp of the grid a block (steps of the paper's size: 15 k rows are 480 blocks of 32 for 2,960 warps).
int aggregate_block_shift(int64_t rows) {
  const int64_t warps = int64_t(kNumSMs) * XRL_AGG_CTAS * TW;
  if ((rows + 31) / 32 >= warps) return 5;
  if ((rows + 15) / 16 >= warps) return 4;
  return 3;
}

namespace {

bool make_row_map(CUtensorMap* m, const void* ptr, CUtensorMapDataType dt, uint32_t elem_bytes,
                  uint64_t rows, uint32_t cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {uint64_t(cols) * elem_bytes};
  cuuint32_t box[2] = {cols, 1};                 // gather4 takes boxes one row high
  cuuint32_t estr[2] = {1, 1};
  return fn(m, dt, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, int K, bool READOUT, bool MERGED, bool SEQ>
int launch_k_seq(const int32_t* rowptr, const int32_t* col, const void* Z, const float* scores, const float* bias,
             void* h_out, Window win, int64_t buf_rows, const int32_t* seg_id, float* partial,
             const int32_t* self_idx, int32_t* status, cudaStream_t st) {
  static bool attr[64] = {};
  const size_t smem = sizeof(WarpSmem<K, MERGED, G, GQ>) * TW;
  if (!ensure_dynamic_smem(k_aggregate_tma<T, K, READOUT, MERGED, SEQ>, int(smem), attr)) return -1;
  constexpr bool is_bf16 = sizeof(T) == 2;
  CUtensorMap mz, ms;
  if (MERGED) {
    if (!make_merged_map(&mz, Z, uint64_t(buf_rows), 512 + 8 * K)) return -1;
    ms = mz;
  } else if (!make_row_map(&mz, Z, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                           sizeof(T), uint64_t(buf_rows), is_bf16 ? 256 : 128) ||
             !make_row_map(&ms, scores, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, uint64_t(buf_rows), 2 * K)) {
    return -1;
  }
  const int64_t rows = int64_t(win.row_end) - win.row_begin;
  const int shift = aggregate_block_shift(rows);
  const int64_t br = int64_t(1) << shift;
  const int64_t nblocks = (rows + br - 1) / br;
  int64_t nb = (rows + br * TW - 1) / (br * TW);
  if (nb > int64_t(kNumSMs) * XRL_AGG_CTAS) nb = int64_t(kNumSMs) * XRL_AGG_CTAS;
  k_aggregate_tma<T, K, READOUT, MERGED, SEQ><<<int(nb), TW * 32, smem, st>>>(
      mz, ms, rowptr, col, static_cast<const T*>(Z), reinterpret_cast<const float2*>(scores), bias,
      static_cast<T*>(h_out), win, seg_id, partial, int32_t(nblocks), self_idx, status, int32_t(shift));
  return 1;
}


template <typename T, int K, bool READOUT, bool MERGED>
int launch_k(const int32_t* rowptr, const int32_t* col, const void* Z, const float* scores, const float* bias,
             void* h_out, Window win, int64_t buf_rows, const int32_t* seg_id, float* partial,
             const int32_t* self_idx, int32_t* status, cudaStream_t st) {
  // launches of fewer than 32 rows per block are the ones the all-layers kernel can stand in for (merged rows only)
  if (MERGED && aggregate_block_shift(int64_t(win.row_end) - win.row_begin) < 5)
    return launch_k_seq<T, K, READOUT, MERGED, MERGED>(rowptr, col, Z, scores, bias, h_out, win, buf_rows, seg_id,
                                                       partial, self_idx, status, st);
  return launch_k_seq<T, K, READOUT, MERGED, false>(rowptr, col, Z, scores, bias, h_out, win, buf_rows, seg_id,
                                                    partial, self_idx, status, st);
}

}  // namespace

// buf_rows: rows of the Z / scores buffers reachable from this window (indices are window-relative).
// partial != nullptr selects the variant fused with the per-graph sum (then h_out is not written and
// the window must start at row 0).  Returns kernels launched, or -1 when this shape is not handled here.
int launch_aggregate_tma(const Dims& d, const int32_t* rowptr, const int32_t* col, const void* Z,
                         const float* scores, const float* bias, void* h_out, Window win, int64_t buf_rows,
                         const int32_t* seg_id, float* partial, int32_t* status, cudaStream_t st,
                         const int32_t* self_idx) {
  if (encode_fn() == nullptr) return -1;
  const bool bf = d.dtype == XRL_BF16 && d.H == 256, fp = d.dtype == XRL_FP32 && d.H == 128;
  if (!bf && !fp) return -1;
  if (d.zmerged && !bf) return -1;
  if (partial != nullptr && (win.row_begin != 0 || win.win_base != 0)) return -1;
#define TMA_ARGS rowptr, col, Z, scores, bias, h_out, win, buf_rows, seg_id, partial, self_idx, status, st
#define TMA_CASE(KK)                                                                                   \
  case KK:                                                                                             \
    if (d.zmerged)                                                                                     \
      return partial ? launch_k<bf16, KK, true, true>(TMA_ARGS) : launch_k<bf16, KK, false, true>(TMA_ARGS); \
    if (partial != nullptr)                                                                            \
      return bf ? launch_k<bf16, KK, true, false>(TMA_ARGS) : launch_k<float, KK, true, false>(TMA_ARGS);    \
    return bf ? launch_k<bf16, KK, false, false>(TMA_ARGS) : launch_k<float, KK, false, false>(TMA_ARGS);
  switch (d.K) {
    TMA_CASE(4) TMA_CASE(8) TMA_CASE(16)
    default: return -1;
  }
#undef TMA_ARGS
#undef TMA_CASE
}

// Shapes this kernel takes (512-byte feature rows, 4 | K).
bool aggregate_tma_shape(const Dims& d) {
  const bool bf = d.dtype == XRL_BF16 && d.H == 256, fp = d.dtype == XRL_FP32 && d.H == 128;
  return (bf || fp) && (d.K == 4 || d.K == 8 || d.K == 16) && encode_fn() != nullptr;
}

// Partial-sum slots the fused variant writes for `rows` rows and B graphs.
// (an upper bound over every row count up to `rows`: small launches use smaller blocks, at most 2 x the warps
// of a full grid of them)
int64_t aggregate_readout_slots(int64_t rows, int64_t B) {
  const int64_t full = (rows + BR - 1) / BR, small = 2 * int64_t(kNumSMs) * XRL_AGG_CTAS * TW;
  return (full > small ? full : small) + B;
}
int32_t aggregate_readout_blocks(int64_t rows) {
  const int shift = aggregate_block_shift(rows);
  return int32_t((rows + (int64_t(1) << shift) - 1) >> shift);
}

}  // namespace xrl

// Internal declarations shared by the kernels and the C-ABI layer of libxrl.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "xrl.h"

namespace xrl {

constexpr int kS = 8;            // shape features per node (compile-time in the kernels)
constexpr int kNumSMs = 148;     // B200
constexpr float kLog2e = 1.4426950408889634f;   // half-scores are stored multiplied by log2(e)

typedef __nv_bfloat16 bf16;

// First error wins; kernels never trap.
__device__ __forceinline__ void raise(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

// ---- 16-byte vectors of the storage type ------------------------------------------------
template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int N = 4; };
template <> struct VecOf<bf16> { static constexpr int N = 8; };

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

__device__ __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
  f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
  f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ uint4 pack(const float (&f)[4]) {
  return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                    __float_as_uint(f[3]));
}
__device__ __forceinline__ uint4 pack(const float (&f)[8]) {
  return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                    pack_bf16x2(f[6], f[7]));
}
template <typename T>
__device__ __forceinline__ void load_vec(const T* p, float (&f)[VecOf<T>::N]) {
  unpack(__ldg(reinterpret_cast<const uint4*>(p)), f);
}
template <typename T>
__device__ __forceinline__ void store_vec(T* p, const float (&f)[VecOf<T>::N]) {
  *reinterpret_cast<uint4*>(p) = pack(f);
}
__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(bf16 x) { return __bfloat162float(x); }

// ---- device-side weights ------------------------------------------------------------------
struct LayerWeights {
  const void* W;        // storage type, [H x H] row-major [in x out]
  const void* Wt;       // bf16 only: transpose [out x in] (K-major B operand of the tensor-core path)
  const float* a_src;   // [H]
  const float* a_dst;   // [H]
  const float* b;       // [H]
};
struct DevWeights {
  const void* W0;       // storage type, [(2S+T) x H]
  const float* b0;
  LayerWeights layer[64];
  const float* Wg; const float* bg;
  const float *pW1, *pb1, *pWh, *pbh, *pw2, *pb2;     // Wh, bh: second hidden layer (Hm2 > 0)
  const float *vW1, *vb1, *vWh, *vbh, *vw2, *vb2;
};

struct Dims {
  int T, H, K, L, Hm, Dg, A;
  int dtype;
  int Hm2;            // second hidden width of the heads' MLPs, 0 = none
  // 1: each row of the Z buffer is followed by the node's K {s_src, s_dst} pairs (row stride
  // H * sizeof(storage) + 8 K bytes), so that one gather brings both; set only when the tensor-core
  // transform and the TMA aggregate kernel handle the shape (the `scores` arguments are then unused)
  int zmerged;
};
inline size_t z_row_bytes(const Dims& d) {
  return size_t(d.H) * (d.dtype == XRL_BF16 ? 2 : 4) + (d.zmerged ? size_t(8) * d.K : 0);
}
bool aggregate_tma_shape(const Dims& d);
// all attention layers of a small step in one cooperative launch (bf16, hidden 256, merged Z rows)
bool layers_coop_supported(const Dims& d, int layers, int64_t rows);
int64_t layers_coop_max_rows();

// Opt-in to large dynamic shared memory is a per-device function attribute: remember it per device.
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, int bytes, bool (&done)[64]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return false; }
  if (done[dev]) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  done[dev] = true;
  return true;
}

// ---- launchers (each returns the number of kernels it launched; errors via cudaGetLastError) --
struct PackIn {
  int32_t B, num_envs, N, E;
  int32_t max_n, max_m;                           // largest node / edge count of one graph
  const int32_t *n_nodes, *n_edges, *env_off;     // device copies of the metadata
  const int32_t *op, *edge_src, *edge_dst;        // device
};
struct PackOut {
  int32_t *node_off, *edge_off, *seg_id, *graph_env, *rowptr, *col;
  int32_t *deg, *tmp_eid /* [2E]: (edge id, producer) pairs */, *long_rows, *long_count, *scan_ws, *coarse;   // scratch
  int32_t* eid = nullptr;   // optional output [E]: the input edge in each CSR slot (attributes on edges)
};
int launch_pack(const PackIn& in, const PackOut& out, int T, int32_t* status, cudaStream_t st);
// the same in two parts, for packing a batch range by range while its later graphs are still being copied
bool pack_per_graph(const PackIn& in);
int launch_pack_offsets(const PackIn& in, const PackOut& out, cudaStream_t st);
int launch_pack_graphs(const PackIn& in, const PackOut& out, int T, int32_t g0, int32_t g1, int32_t* status,
                       cudaStream_t st, bool offsets = false);
size_t scan_workspace_ints(int64_t n);
int launch_merge_csr(const int32_t* rp_a, const int32_t* col_a, const int32_t* rp_b, const int32_t* col_b,
                     int32_t N, int32_t* rp_m, int32_t* col_m, cudaStream_t st);
int launch_permute_edge_rows(const void* src, const int32_t* eid, void* dst, int64_t E, int row_bytes,
                             cudaStream_t st);
// out[0..n_in] = exclusive prefix sums of in[0..n_in) (n_in + 1 outputs); ws: scan_workspace_ints(n_in) ints
int launch_exclusive_scan(const int32_t* in, int32_t* out, int32_t n_in, int32_t* ws, cudaStream_t st);

// Row lists (delta encoding): `row_list` makes the node-update kernels read node row_list[r] and write
// row r of a dense buffer; `self_idx` tells the aggregate kernels where row r's own Z row lives (its
// producers come from the compact CSR it is given).
// Row windows: kernels process global rows [row_begin, row_end); activation buffers (h, Z,
// scores) are indexed by (row - win_base), CSR / op / shape arrays by the global row id.
struct Window { int32_t row_begin, row_end, win_base; };

// eattr (optional, [E x S] storage type, CSR slot order): Eq. 6 sums these instead of the producers' shapes
int launch_embed(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op,
                 const void* shape, const DevWeights& w, void* h, Window win, cudaStream_t st,
                 const int32_t* row_list = nullptr, const void* eattr = nullptr);
// scores: [N][K] pairs {s_src, s_dst} (float2), both already multiplied by log2(e)
int launch_xform_simt(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
                      Window win, cudaStream_t st);
bool embed_umma_supported(const Dims& d);
int embed_umma_kpad(const Dims& d);
void build_w0ext(const Dims& d, const void* W0_store, const float* b0, void* out, cudaStream_t st);
int launch_embed_umma(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op,
                      const void* shape, const void* w0ext_t, void* h, Window win, int32_t* status,
                      cudaStream_t st, const int32_t* row_list = nullptr, const void* eattr = nullptr);
bool xform_umma_supported(const Dims& d);
int launch_xform_umma(const Dims& d, const void* h, const LayerWeights& lw, void* Z, float* scores,
                      Window win, int32_t* status, cudaStream_t st);
int launch_scores(const Dims& d, const void* Z, const LayerWeights& lw, float* scores, Window win,
                  cudaStream_t st);
int launch_aggregate(const Dims& d, const int32_t* rowptr, const int32_t* col, const void* Z,
                     const float* scores, const float* bias, void* h_out,
                     Window win, int64_t buf_rows, int32_t* status, cudaStream_t st,
                     const int32_t* self_idx = nullptr);
int launch_aggregate_tma(const Dims& d, const int32_t* rowptr, const int32_t* col, const void* Z,
                         const float* scores, const float* bias, void* h_out, Window win, int64_t buf_rows,
                         const int32_t* seg_id, float* partial, int32_t* status, cudaStream_t st,
                         const int32_t* self_idx = nullptr);
// h is read and overwritten; Z0 / Z1: two buffers of `rows` merged Z rows; partial != nullptr: the last layer leaves
// the per-block sums of Eq. 8 instead of node features; sync: two zeroed words only this kernel touches.
// Returns kernels launched or -1 (not handled / refused).
int launch_layers_coop(const Dims& d, const DevWeights& dw, int layers, void* h, void* Z0, void* Z1,
                       const int32_t* rowptr, const int32_t* col, int64_t rows, const int32_t* seg_id,
                       float* partial, int32_t* status, uint32_t* sync, cudaStream_t st);
int aggregate_block_shift(int64_t rows);           // log2(rows per block) the TMA aggregate uses for `rows` rows
int64_t aggregate_readout_slots(int64_t rows, int64_t B);
int32_t aggregate_readout_blocks(int64_t rows);
// block_shift: aggregate_block_shift of the launch that wrote `partial`
int launch_global_update_blocks(const Dims& d, const float* partial, const int32_t* node_off, int32_t nblocks,
                                int block_shift, const float* g0, const DevWeights& w, float* emb, int32_t B,
                                cudaStream_t st);
int launch_readout(const Dims& d, const void* h, const int32_t* chunk_row0, const int32_t* chunk_row1,
                   int32_t chunk_begin, int32_t chunk_end, float* partial, int32_t win_base,
                   cudaStream_t st, const int32_t* remap = nullptr);

// ---- delta encoding: candidates reuse the rows of their environment's current graph ---------------
struct DeltaIn {
  int32_t N, E;
  const int32_t *seg_id, *graph_env, *env_off, *node_off, *rowptr, *col, *op;
  const void* shape;
  int shape_bytes;                 // bytes of one node's shape features
  const int32_t* base_id;          // caller's hint
};
int launch_delta_level0(const DeltaIn& in, int32_t* valid, int32_t* base, int32_t* level, cudaStream_t st);
int launch_delta_propagate(const DeltaIn& in, int32_t t, const int32_t* level_in, int32_t* level_out,
                           cudaStream_t st);
int launch_delta_count(int32_t N, int32_t L, const int32_t* level, int32_t* counts, int32_t* cursor,
                       cudaStream_t st);
int launch_delta_assign(int32_t N, int32_t L, const int32_t* level, const int32_t* counts, int32_t* cursor,
                        int32_t* rank, int32_t* list, cudaStream_t st);
int launch_delta_degrees(const DeltaIn& in, int32_t n, const int32_t* list, int32_t* deg, cudaStream_t st);
int launch_delta_fill(const DeltaIn& in, int32_t n, int32_t t, const int32_t* list, const int32_t* rowptr_c,
                      const int32_t* level, const int32_t* rank, const int32_t* base, int32_t* col_c,
                      int32_t* self_c, cudaStream_t st);
int launch_delta_remap(int32_t N, int32_t L, const int32_t* level, const int32_t* rank, const int32_t* base,
                       int32_t* remap, cudaStream_t st);
int launch_global_update(const Dims& d, const float* partial, const int32_t* graph_chunk_off,
                         const float* g0, const DevWeights& w, float* emb, int32_t B, cudaStream_t st);
int launch_heads(const Dims& d, const DevWeights& w, const float* emb, const int32_t* env_off,
                 const uint8_t* mask, int32_t B, int32_t num_envs, float* logit_ws, float* probs,
                 float* value, int32_t* action, uint64_t seed, uint64_t step, int32_t* status,
                 cudaStream_t st);
int launch_sample(const float* probs, int32_t num_envs, int32_t A1, uint64_t seed, uint64_t step,
                  int32_t* action, cudaStream_t st);
// ---- reverse pass (Section 3.3.4) --------------------------------------------------------------------
size_t ppo_heads_workspace_floats(const Dims& d, int64_t B, int64_t num_envs);
int launch_ppo_heads(const Dims& d, const DevWeights& w, float* grad_base, const float* w_base, const void* hL,
                     const int32_t* node_off, const int32_t* seg_id, const float* g0, const int32_t* env_off,
                     const uint8_t* mask, const int32_t* action, const float* logp_old, const float* adv,
                     const float* ret, float eps, float c1, float c2, int32_t B, int32_t num_envs, int64_t N,
                     float* ws, float* loss, float* dh, float* logp_out, int32_t* status, cudaStream_t st);
int launch_gat_layer_bwd(const Dims& d, const int32_t* rowptr, const int32_t* col, const void* Z, const float* scores,
                         const void* h_in, const void* h_out, const float* dh_out, float* dh_in, float* dz,
                         float* ds, void* dz_store, const LayerWeights& lw, float* gW, float* ga_src, float* ga_dst,
                         float* gb, int32_t N, cudaStream_t st);
int launch_gae(const float* reward, const float* values, const uint8_t* done, float gamma, float lambda, int32_t T,
               int32_t M, float* adv, float* ret, cudaStream_t st);
int launch_grad_weigh(int elem_bytes, const void* grad, int64_t count, const void* loss, int64_t n, void* buf,
                      cudaStream_t st);
int launch_grad_unweigh(int elem_bytes, const void* buf, int64_t count, void* grad, void* loss, cudaStream_t st);
size_t embed_bwd_smem_bytes(const Dims& d);
int launch_embed_bwd(const Dims& d, const int32_t* rowptr, const int32_t* col, const int32_t* op, const void* shape,
                     const void* eattr, const void* h0, const float* dh0, float* xs /* scratch [N x 16] */,
                     float* gW0, float* gb0, int32_t N, cudaStream_t st);
int launch_init_weights(float* blob, int64_t first, int64_t count, float bound, uint64_t seed, cudaStream_t st);
int launch_to_float(const void* src, int dtype, float* dst, int64_t n, cudaStream_t st);
int launch_round_weights(const float* src, void* dst, void* dst_t, int rows, int cols, int dtype,
                         cudaStream_t st);

}  // namespace xrl

/* xrl -- the per-step forward pass of the X-RLflow agent on one NVIDIA B200 (sm_100a).
 *
 * At every rewrite step the agent observes the current computation graph together with all
 * of its candidate rewritten graphs, encodes them with a graph neural network, reads out one
 * vector per graph and evaluates an actor-critic policy head (masked categorical distribution
 * over the candidates plus No-Op) and a value head (paper Sections 3.3.2, 3.3.3 and 3.4).
 * This library is that path and nothing else:
 *
 *     xrl_pack / xrl_pack_flat   Section 3.3.2  batch the graphs into one meta-graph (CSR)
 *     xrl_encode                 Section 3.4    Eq. 6 -> L x Eq. 7 -> Eq. 8
 *     xrl_policy_value           Section 3.3.2  policy / value MLPs, padded action space,
 *                                Section 3.3.3  invalid-action masking, No-Op, sampling
 *     xrl_ppo_grad, xrl_gae      Section 3.3.4  the training step's objective (Eq. 3-5) and its gradient with
 *                                               respect to every weight; advantage estimates
 *
 * Conventions
 *  - Plain C ABI.  Every function returns an xrl_status; nothing throws, aborts or traps.
 *  - "host" / "device" on every pointer says where the memory lives.  The caller owns every
 *    buffer it passes in; the library owns xrl_ctx and xrl_batch objects.
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default stream)
 *    and is asynchronous.  Argument errors are returned before anything is enqueued.  Errors
 *    found by kernels (malformed graph ids, bad masks, bounded waits that ran out) are written
 *    to a device status word; read it with xrl_last_device_status after the stream is synced.
 *  - A context is bound to one device and is not thread-safe; distinct contexts are independent.
 *  - There is no CPU fallback: without a CUDA device xrl_create fails with XRL_ERR_CUDA.
 *
 * Readings of what the paper leaves open: ReLU for every sigma; LeakyReLU(0.2) inside the
 * attention score (the GAT paper's choice); neighbourhood = producers of the node plus the
 * node itself; K heads of width H/K concatenated in every layer; a bias in every dense map;
 * Eq. 8 carries a weight matrix W_g; the policy scores each graph with one shared MLP and the
 * current graph's score is the No-Op logit.
 */
#ifndef XRL_H_
#define XRL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t xrl_status;
enum {
  XRL_OK = 0,
  XRL_ERR_INVALID_ARG = 1, /* null pointer, negative size, inconsistent offsets, bad mask  */
  XRL_ERR_BAD_GRAPH = 2,   /* edge endpoint outside [0, num_nodes), self edge, op id >= T   */
  XRL_ERR_CAPACITY = 3,    /* batch larger than the capacities given to xrl_create          */
  XRL_ERR_ALLOC = 4,       /* host or device allocation failed                              */
  XRL_ERR_CUDA = 5,        /* a CUDA runtime call failed (also: no device)                  */
  XRL_ERR_STATE = 6,       /* weights not set, batch not packed, batch of another context   */
  XRL_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out                            */
  XRL_ERR_UNSUPPORTED = 8  /* model shape outside what the kernels are built for            */
};

enum { XRL_FP32 = 0, XRL_BF16 = 1 };      /* storage type of features / Eq. 6-7 weights      */
enum { XRL_MEM_HOST = 0, XRL_MEM_DEVICE = 1 };

/* Model and capacity description (plain data, copied by xrl_create).
 * Supported shapes: hidden a multiple of 32 in [32, 512]; hidden / heads a multiple of 8;
 * num_shape_feats = 8; num_op_types <= 256; mlp_hidden in [1, 1024]; mlp_hidden2 in [0, 1024];
 * global_dim in [0, 16]. */
typedef struct {
  int32_t num_op_types;    /* T: size of the operator table (one-hot node attribute)          */
  int32_t num_shape_feats; /* S: shape features per node (attribute of its outgoing edges)    */
  int32_t hidden;          /* H                                                               */
  int32_t heads;           /* K, must divide H                                                */
  int32_t layers;          /* L: number of graph-attention layers (the paper's k), >= 0       */
  int32_t mlp_hidden;      /* Hm: (first) hidden width of the policy and value MLPs           */
  int32_t mlp_hidden2;     /* Hm2: second hidden width, 0 = none.  Section 3.3.2 describes the heads
                              as two-layer MLPs, the hyper-parameter table lists hidden sizes
                              [256, 64]: (Hm, Hm2) = (256, 64) is that table's model, Hm2 = 0 the
                              one-hidden-layer reading                                             */
  int32_t global_dim;      /* Dg: width of the per-graph global attribute (paper: value 0)    */
  int32_t dtype;           /* XRL_FP32, or XRL_BF16 = bf16 storage with fp32 accumulation     */
  int32_t edge_attributes; /* 0: the attribute of edge j -> i in Eq. 6 is producer j's S shape features
                              (taken from `shape`); 1: every edge has S attributes of its own, given with
                              xrl_batch_set_edge_attr after packing - Section 3.3.2 as written, where an
                              edge carries the shape of its tensor divided by the constant M             */
  int32_t neighbourhood;   /* Eq. 7's neighbours of a node: 0 = its producers (and itself), 1 = its
                              producers and its consumers (and itself) - "neighbours" read both ways;
                              Eq. 6 sums over incoming edges either way.  With 1 the packer also
                              builds the CSR by producer and a merged one (8 more bytes per edge and
                              node), large batches are not packed range by range, and
                              xrl_encode_delta is not available (XRL_ERR_UNSUPPORTED)            */
  int32_t max_actions;     /* A_max: padded number of candidate slots; No-Op is index A_max   */
  int32_t max_graphs;      /* capacity: graphs per batch                                      */
  int32_t max_envs;        /* capacity: environments per batch                                */
  int64_t max_nodes;       /* capacity: total nodes per batch (< 2^31)                        */
  int64_t max_edges;       /* capacity: total edges per batch (< 2^31)                        */
} xrl_model_config;

/* One computation graph: nodes are tensor operators, an edge (src -> dst) is a tensor produced
 * by src and consumed by dst.  All pointers HOST, read-only to the library. */
typedef struct {
  int32_t num_nodes, num_edges;
  const int32_t* op;       /* [num_nodes]      operator id in [0, T)                           */
  const void* shape;       /* [num_nodes x S]  float (XRL_FP32) or bf16 bits (XRL_BF16)        */
  const int32_t* edge_src; /* [num_edges]      producer, local id                              */
  const int32_t* edge_dst; /* [num_edges]      consumer, local id; src != dst; repeats allowed */
} xrl_graph;

typedef struct xrl_ctx xrl_ctx;
typedef struct xrl_batch xrl_batch;

/* ---- context and weights -------------------------------------------------------------- */

/* Create a context on CUDA device `device`: validates the config, allocates the activation
 * workspace for the stated capacities: two feature buffers of max_nodes * H * sizeof(storage) bytes,
 * 8 * heads bytes of half-scores per node, 4 * H bytes of readout partial sums per 32 nodes (the first
 * xrl_encode_delta call adds about 40 bytes per node and 4 per edge).  *out is HOST.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA, ALLOC. */
xrl_status xrl_create(const xrl_model_config* cfg, int32_t device, xrl_ctx** out);
void xrl_destroy(xrl_ctx* ctx);

/* Size in bytes of the flat fp32 weight blob.  Order (matrices row-major [in x out]):
 *   W0 [(S+T+S) x H], b0 [H]                       Eq. 6; input = [edge aggregate | one-hot op | own shape]
 *   per layer: W [H x H], a_src [H], a_dst [H], b [H]   Eq. 7; a_* are K per-head vectors of width H/K
 *   Wg [(H+Dg) x H], bg [H]                        Eq. 8; input = [node sum | global attribute]
 *   policy: W1 [H x Hm], b1 [Hm], (Wh [Hm x Hm2], bh [Hm2] when Hm2 > 0), w2 [last hidden width], b2 [1]
 *   value:  W1 [2H x Hm], b1 [Hm], (Wh, bh likewise), w2 [last hidden width], b2 [1]
 *           input = [current graph | mean of valid candidates]
 *   A head computes w2 . ReLU(Wh^T ReLU(W1^T x + b1) + bh) + b2, without the middle map when Hm2 = 0. */
xrl_status xrl_weights_size(const xrl_ctx* ctx, size_t* bytes);
/* Upload the blob (HOST, fp32).  With XRL_BF16 the library rounds W0 and the layer matrices W
 * to bf16 (nearest even) once; everything else stays fp32.  Synchronous. */
xrl_status xrl_set_weights(xrl_ctx* ctx, const void* host_blob, size_t bytes);
/* Read the fp32 blob back (HOST, same layout and size; the master copy, not the bf16-rounded one):
 * together with xrl_set_weights this is the checkpoint / restore of a model.  Synchronous. */
xrl_status xrl_get_weights(const xrl_ctx* ctx, void* host_blob, size_t bytes);

/* Seeded initial weights in place of xrl_set_weights (the paper names no initialisation; Xavier-uniform is
 * this library's choice): matrices U(-b, b) with b = sqrt(6 / (fan_in + fan_out)), the attention vectors with
 * fan (H / heads, 1), the heads' last layers with fan (hidden, 1), every bias U(-0.1, 0.1).  Element i of the
 * blob is b * ((w >> 8) * 2^-23 - 1), w = first word of Philox4x32-10 with key = seed and counter (i, 0, 0, 1):
 * reproducible bit for bit from the seed on any device.  Synchronises the device.  Errors: INVALID_ARG, CUDA. */
xrl_status xrl_init_weights(xrl_ctx* ctx, uint64_t seed);

/* ---- (1) packer: Section 3.3.2, the current graph and its candidates become one meta-graph ---- */

/* graphs[env_off[e]] is the CURRENT graph of environment e and graphs[env_off[e]+1 ..
 * env_off[e+1]-1] are its candidates in action order.  env_off is HOST, [num_envs + 1],
 * env_off[0] = 0, strictly increasing, env_off[num_envs] = num_graphs.
 * The batch holds, on the device: node_off[B+1], edge_off[B+1] (exclusive prefix sums),
 * seg_id[N] (node -> graph), graph_env[B], CSR by consumer rowptr[N+1] / col[E] over global
 * node ids (inside a row the producers keep the order of the input edge list), op[N],
 * shape[N x S].  If *out is NULL a batch sized to the context's capacities is allocated;
 * otherwise the existing batch is re-packed in place with no allocation.
 * Graph validity (ids in range, no self edge, op < T) is checked on the device: a violation
 * sets XRL_ERR_BAD_GRAPH in the device status word; the offending edges are left out and the slots
 * they would have taken are filled with a valid node id, so encoding such a batch anyway reads only
 * inside the arrays (nothing faults), but its results describe no graph the caller gave: read the
 * status word before trusting them. */
xrl_status xrl_pack(xrl_ctx* ctx, const xrl_graph* graphs, int32_t num_graphs,
                    const int32_t* env_off, int32_t num_envs, void* stream, xrl_batch** out);

/* Same operation on already concatenated arrays.  n_nodes, n_edges [num_graphs] and env_off
 * are always HOST; op [N], shape [N x S], edge_src [E], edge_dst [E] (local ids, graphs back
 * to back) are HOST or DEVICE according to `where` (XRL_MEM_*).  DEVICE arrays are read by the
 * kernels directly and must stay valid until the stream has passed the call.  HOST arrays in
 * pageable memory are staged through a pinned buffer before the call returns; HOST arrays that are
 * all page-locked (cudaHostAlloc / cudaHostRegister) are copied asynchronously straight from the
 * caller's memory and must then also stay valid until the stream has passed the call.
 * A page-locked batch of 2^20 nodes or more (graphs of at most 16,384 nodes) is copied and packed in
 * up to 8 ranges of whole graphs on a stream the batch owns, ordered after everything queued on `stream`
 * so far; xrl_encode then encodes range after range as each arrives (graphs never interact before the
 * heads), so that the bus transfer of the later ranges overlaps the encoding of the earlier ones.  Every
 * other consumer of the batch first waits for all ranges; results do not depend on the split except for
 * the order in which a graph's node features are summed (Eq. 8), i.e. within rounding.  The host arrays of
 * such a batch are read by that stream: keep them valid until a consumer of the batch queued after this
 * call (xrl_encode, ...) has completed on its stream, or until xrl_last_device_status has returned. */
xrl_status xrl_pack_flat(xrl_ctx* ctx, int32_t where, int32_t num_graphs, const int32_t* n_nodes,
                         const int32_t* n_edges, const int32_t* op, const void* shape,
                         const int32_t* edge_src, const int32_t* edge_dst, const int32_t* env_off,
                         int32_t num_envs, void* stream, xrl_batch** out);

xrl_status xrl_batch_free(xrl_ctx* ctx, xrl_batch* batch);
/* All four outputs HOST. */
xrl_status xrl_batch_info(const xrl_batch* batch, int64_t* num_nodes, int64_t* num_edges,
                          int32_t* num_graphs, int32_t* num_envs);
/* Copy the packed index arrays to HOST buffers (any may be NULL); synchronises the stream the
 * batch was packed on.  Sizes: rowptr [N+1], col [E], seg_id [N], node_off [B+1],
 * edge_off [B+1], graph_env [B]. */
xrl_status xrl_batch_export(const xrl_batch* batch, int32_t* rowptr, int32_t* col, int32_t* seg_id,
                            int32_t* node_off, int32_t* edge_off, int32_t* graph_env);

/* Attributes on the edges (contexts created with edge_attributes = 1; Section 3.3.2: an edge's attribute is
 * the shape of the tensor it carries, padded to rank 4 and divided by a constant).  edge_attr is
 * [E x S] in the storage type (float, or bf16 bits), one row per edge in the order of the edge lists given
 * to the pack call, HOST or DEVICE according to `where`; the library brings the rows into the order of the
 * packed CSR (one gather pass, queued on `stream` after the packing) and Eq. 6 then sums, for each node, the
 * attributes of its incoming edges in place of its producers' shape features.  Call it after every pack of
 * the batch and before xrl_encode (which returns XRL_ERR_STATE otherwise).  A HOST array is read before the
 * call returns.  xrl_encode_delta is not available for such contexts (XRL_ERR_UNSUPPORTED).
 * Errors: INVALID_ARG, STATE (context without edge attributes, batch not packed, recording), CUDA. */
xrl_status xrl_batch_set_edge_attr(xrl_ctx* ctx, xrl_batch* batch, int32_t where, const void* edge_attr,
                                   void* stream);

/* ---- (2) encoder: Section 3.4 ------------------------------------------------------------ */

/* Eq. 6:  h0_i = ReLU(W0^T [ sum_{j -> i} shape_j | onehot(op_i) | shape_i ] + b0)
 * Eq. 7 (L times):  z = W^T h;  e_ij = LeakyReLU_0.2(a_src . z_j + a_dst . z_i) per head over
 *         j in producers(i) + {i};  alpha = softmax_j e_ij;  h'_i = ReLU(sum_j alpha_ij z_j + b)
 * Eq. 8:  emb_g = ReLU(Wg^T [ sum_{i in g} h_i | g0_g ] + bg)
 * g0: DEVICE fp32 [B x Dg] or NULL (= 0, the paper's initial value).
 * graph_emb: DEVICE fp32 [B x H], written by the call. */
xrl_status xrl_encode(xrl_ctx* ctx, const xrl_batch* batch, const float* g0, float* graph_emb,
                      void* stream);

/* Delta encoding: same result as xrl_encode (within rounding), computed only where it can differ.
 * The candidates of a step are the current graph with one rewrite applied at one location (paper
 * Sections 3.2, 3.3.1), so almost every candidate node equals a node of the current graph.  A candidate
 * node with the same operator, shape features and producers as a current-graph node, whose producers are
 * unchanged too, has that node's features after Eq. 6; a change reaches a node one attention layer after
 * it reached one of its producers (Eq. 7 looks at producers only).  Per layer the library lists the rows
 * a change has reached, runs the encoder kernels on those rows only (current graphs are always computed
 * in full) and lets every other candidate node read its current-graph twin.
 *   base_id  DEVICE int32 [N], or NULL: for node i of a candidate graph, the global (packed) id of the node
 *            of its environment's current graph that it corresponds to, or -1.  It is a HINT: the library
 *            verifies operator, shape features and producer lists on the device and recomputes whatever
 *            does not check out, so a wrong hint costs time, never correctness.  Entries of current-graph
 *            nodes are ignored.
 * The call synchronises `stream` once (it reads the number of rows per layer back).
 * xrl_delta_rows reports, for the last call, the rows computed at Eq. 6 and after each attention layer
 * (HOST int64 [count], count <= L + 1). */
xrl_status xrl_encode_delta(xrl_ctx* ctx, const xrl_batch* batch, const int32_t* base_id, const float* g0,
                            float* graph_emb, void* stream);
xrl_status xrl_delta_rows(const xrl_ctx* ctx, int64_t* rows, int32_t count);

/* Debug aid for parity tests: run Eq. 6 and the first `num_layers` attention layers
 * (0 <= num_layers <= L) and copy the node features to HOST fp32 [N x H].  Synchronous. */
xrl_status xrl_debug_node_features(xrl_ctx* ctx, const xrl_batch* batch, int32_t num_layers,
                                   float* host_out, void* stream);

/* ---- (3) heads: Sections 3.3.2 and 3.3.3 -------------------------------------------------- */

/* Per graph g: logit_g = w2 . ReLU(W1^T emb_g + b1) + b2 (policy MLP).  Per environment e with
 * C candidates: action a < C is candidate a, action A_max is No-Op and takes the current graph's
 * logit; probs = softmax over { a : mask[e][a] = 1 } + { No-Op }, every other entry exactly 0.
 * value_e = value MLP of [ emb(current) | mean of emb over the valid candidates ] (zero vector
 * if there is none).
 *   graph_emb DEVICE fp32 [B x H]            (the output of xrl_encode)
 *   mask      DEVICE u8  [num_envs x A_max]  1 = valid; a set bit at a >= C raises
 *                                            XRL_ERR_INVALID_ARG in the device status word
 *   probs     DEVICE fp32 [num_envs x (A_max+1)], last column = No-Op
 *   value     DEVICE fp32 [num_envs]
 *   action    DEVICE int32 [num_envs], or NULL for no sampling.  The draw uses Philox4x32-10
 *             keyed by `seed` with counter (env, step lo, step hi, 0): r = word0 | word1 << 32;
 *             q_a = floor(p_a * 2^32); t = floor(r * sum(q) / 2^64); action = first index whose
 *             inclusive prefix sum of q exceeds t (No-Op if sum(q) = 0).  Integer-exact given
 *             the fp32 probabilities. */
xrl_status xrl_policy_value(xrl_ctx* ctx, const xrl_batch* batch, const float* graph_emb,
                            const uint8_t* mask, float* probs, float* value, int32_t* action,
                            uint64_t seed, uint64_t step, void* stream);

/* The sampling step alone on caller-supplied probabilities: probs DEVICE fp32
 * [num_envs x num_actions] -> action DEVICE int32 [num_envs]; same draw as above. */
xrl_status xrl_sample(xrl_ctx* ctx, const float* probs, int32_t num_envs, int32_t num_actions,
                      uint64_t seed, uint64_t step, int32_t* action, void* stream);

/* ---- (4) the training step's gradient: Section 3.3.4 -------------------------------------------- */

/* The PPO objective over the environments of a packed batch, each a stored transition (its observation =
 * the environment's graphs, the action taken, the behaviour policy's log-probability of it, its advantage
 * estimate and its value target), and the gradient of that objective with respect to every weight:
 *   ratio_e  = exp(log pi(action_e) - logp_old_e)
 *   L_clip   = - mean_e min(ratio_e adv_e, clip(ratio_e, 1 - eps, 1 + eps) adv_e)         (Eq. 3)
 *   L_vf     =   mean_e (value_e - ret_e)^2                                                (Eq. 4)
 *   L_ent    =   mean_e sum_a p_a log p_a      (minus the policy's entropy)
 *   J        =   L_clip + c1 L_vf + c2 L_ent                                               (Eq. 5)
 * The forward pass is that of xrl_encode and xrl_policy_value with every layer's input and Z kept; the reverse
 * pass runs layer by layer in fp32 (ReLU'(0) = 0, LeakyReLU'(0) = 0.2; where the clipped term of Eq. 3 is
 * the smaller one its slope is zero).  For a bf16 model the gradient of W0 and of the layer matrices is the
 * one with respect to the stored (rounded) values.  Sums over rows use floating-point atomics: the last
 * bits of a gradient may differ from run to run.
 *   g0        DEVICE fp32 [B x Dg] or NULL            mask      DEVICE u8 [num_envs x A_max]
 *   action    DEVICE int32 [num_envs]  in [0, A_max], A_max = No-Op; an action the mask excludes raises
 *                                      XRL_ERR_INVALID_ARG in the device status word (results undefined)
 *   logp_old, adv, ret   DEVICE fp32 [num_envs]
 *   loss_out  DEVICE fp32 [4] = { J, L_clip, L_vf, L_ent }
 *   grad      DEVICE fp32, laid out like the weight blob (xrl_weights_size bytes), overwritten
 *   logp_out  DEVICE fp32 [num_envs] or NULL: log pi(action_e) under the current weights
 * The first call allocates the workspace for the context's capacities ((L + 2) copies of the node features,
 * L of the transformed features Z and three fp32 ones) and therefore synchronises; later calls only enqueue.  Not recordable
 * (XRL_ERR_STATE between xrl_graph_begin and xrl_graph_launch).  XRL_ERR_UNSUPPORTED when
 * (T + 8) x H floats exceed one SM's shared memory (227 KB): the operator block of W0's gradient and a tile
 * of eight rows are kept there.
 * Errors: INVALID_ARG, STATE, UNSUPPORTED, ALLOC, CUDA. */
xrl_status xrl_ppo_grad(xrl_ctx* ctx, const xrl_batch* batch, const float* g0, const uint8_t* mask,
                        const int32_t* action, const float* logp_old, const float* adv, const float* ret,
                        float eps, float c1, float c2, float* loss_out, float* grad, float* logp_out,
                        void* stream);

/* Generalised advantage estimation, the estimator Section 3.3.4 takes its advantages from, for M trajectories of
 * T steps each, stored step-major:
 *   delta_t = r_t + gamma V_{t+1} (1 - done_t) - V_t,   A_t = delta_t + gamma lambda (1 - done_t) A_{t+1},
 *   R_t = A_t + V_t  (the value target of Eq. 4).
 *   reward DEVICE fp32 [T x M]; values DEVICE fp32 [(T + 1) x M] (the last row bootstraps the tail);
 *   done DEVICE u8 [T x M] (1 = the episode ended with step t); adv, ret DEVICE fp32 [T x M].
 * One thread per trajectory.  Needs no context.  Errors: INVALID_ARG, CUDA. */
xrl_status xrl_gae(int32_t device, int32_t num_steps, int32_t num_trajectories, const float* reward,
                   const float* values, const uint8_t* done, float gamma, float lambda, float* adv, float* ret,
                   void* stream);

/* Data-parallel training step (Section 3.3.4: the objective is a mean over the environments of the mini-batch;
 * the paper leaves training on several devices as future work).  Every rank has run xrl_ppo_grad on its own
 * environments, so its gradient and loss terms are means over n_r local environments.  The mean over all
 * ranks' environments is sum_r(n_r x_r) / sum_r(n_r): xrl_grad_weigh writes
 *   buf = [ grad * n | loss[0..3] * n | n ]         (count + 5 elements)
 * for the caller's SUM all-reduce of buf (NCCL, gloo, ... - the collective itself is the caller's), and
 * xrl_grad_unweigh divides the reduced buffer by its last element and writes grad and loss back, which then
 * equal one xrl_ppo_grad call on the concatenation of all ranks' batches.
 *   where       XRL_MEM_DEVICE: all pointers DEVICE, work enqueued on `stream` of `device`;
 *               XRL_MEM_HOST: all pointers HOST, done before the call returns (`device`, `stream` ignored)
 *   elem_bytes  4 (float, what xrl_ppo_grad produces) or 8 (double)
 *   total_envs  HOST or NULL: receives sum_r(n_r); for DEVICE buffers a non-NULL pointer synchronises `stream`
 * Errors: INVALID_ARG, CUDA. */
xrl_status xrl_grad_weigh(int32_t where, int32_t device, int32_t elem_bytes, const void* grad, int64_t count,
                          const void* loss, int64_t num_envs, void* buf, void* stream);
xrl_status xrl_grad_unweigh(int32_t where, int32_t device, int32_t elem_bytes, const void* buf, int64_t count,
                            void* grad, void* loss, int64_t* total_envs, void* stream);

/* Read and clear the device status word.  Synchronises `stream`.  *status (HOST) receives the
 * first error code any kernel recorded since the last call, or XRL_OK. */
xrl_status xrl_last_device_status(xrl_ctx* ctx, void* stream, int32_t* status);

/* ---- one submission per step ------------------------------------------------------------------- */

/* A step of the paper's size (13-50 candidates of a few hundred to a few thousand operators, 5 attention
 * layers) is some twenty kernels of 2-15 microseconds each: launched one by one, the host's per-launch cost
 * (about 6 microseconds) is what bounds the step.  Between xrl_graph_begin and xrl_graph_launch the calls
 * xrl_encode, xrl_policy_value and xrl_sample on this context do not launch anything: their kernels are
 * recorded (stream capture on a stream the context owns; the `stream` arguments of those calls are ignored).
 * xrl_graph_launch turns the record into an executable CUDA graph - the first time by instantiating it, later
 * by updating the previous executable in place, which works as long as the sequence of kernels is the same
 * (sizes, pointers and launch shapes may all differ) - and submits it to `stream` with one call.
 * Results, ordering on `stream` and error reporting are those of the direct calls.
 * xrl_pack*, xrl_encode_delta (which reads sizes back) and the profiling calls are not recordable:
 * they return XRL_ERR_STATE between begin and launch; so does a second xrl_graph_begin.  On any error
 * inside the bracket call xrl_graph_launch all the same (it ends the recording) and discard its result.
 * Errors: INVALID_ARG, STATE (no recording in progress / profiling enabled), CUDA. */
xrl_status xrl_graph_begin(xrl_ctx* ctx);
xrl_status xrl_graph_launch(xrl_ctx* ctx, void* stream);

/* Names of the kernels launched by the last xrl_encode / xrl_policy_value / xrl_pack call on
 * this context and how many launches each call made (HOST outputs, any may be NULL). */
xrl_status xrl_launch_counts(const xrl_ctx* ctx, int64_t* pack, int64_t* encode, int64_t* heads);

/* ---- packing for callers that must not allocate ------------------------------------------------ */

/* (No counterpart in the paper: this is a deployment variant of the packer above.)
 *
 * Some programs that embed this library are not allowed to ask CUDA for memory while they run:
 * an inference server whose own pool already holds the whole GPU (a cudaMalloc there fails, or
 * stalls every stream while the driver synchronises the device), a control loop with a latency
 * budget that a device-wide synchronisation would break, or a plug-in whose host forbids driver
 * allocations from callbacks.  xrl_create / xrl_pack allocate (context workspace, batch, pinned
 * staging), so those programs cannot use them.  This call builds the same packed index arrays
 * with NO allocation of any kind: no context, no batch object, and the packer's scratch (in-degree
 * counters, row cursors, the unsorted (edge id, producer) slots, scan partial sums, a device copy of
 * the counts)
 * sits in a fixed array inside the library image, about 4.8 MB that every GPU loading the library
 * keeps until the process exits.  The price is a size limit:
 *     num_graphs <= XRL_STATIC_PACK_MAX_GRAPHS, num_envs <= XRL_STATIC_PACK_MAX_ENVS,
 *     total nodes <= XRL_STATIC_PACK_MAX_NODES, total edges <= XRL_STATIC_PACK_MAX_EDGES;
 * anything larger is refused with XRL_ERR_CAPACITY before any work is queued (the paper's own
 * steps, 13-50 candidates of a few hundred to a few thousand operators, fit).
 *
 * Arguments: n_nodes, n_edges [num_graphs] and env_off [num_envs + 1] are HOST; they are validated
 * before the call returns and copied to the device with an asynchronous copy on `stream` (ordinary
 * pageable arrays are fully read by then; page-locked arrays must stay unchanged until the stream has
 * passed the call); op [N], edge_src [E], edge_dst [E] are DEVICE inputs with the meaning they have
 * in xrl_pack_flat; node_off [B+1], edge_off [B+1], seg_id [N], graph_env [B], rowptr [N+1],
 * col [E] and device_status [1] are DEVICE outputs owned by the caller.  device_status receives
 * XRL_OK or XRL_ERR_BAD_GRAPH once the stream has run the work.  `device` is the CUDA device the
 * pointers belong to; the call makes it current.
 *
 * The first call on each device looks up the device address of the built-in array once
 * (cudaGetSymbolAddress); make that first call before you begin any stream capture, and from one
 * thread only (first calls on the same device must not run concurrently).  All calls on
 * a device share the one array and it keeps whatever the previous call left there (the kernels
 * re-zero the counters they need), so two calls must never overlap on the GPU: issue them on one
 * stream, or order them with events.  Overlapping calls race and corrupt each other's result. */
#define XRL_STATIC_PACK_MAX_GRAPHS 4096
#define XRL_STATIC_PACK_MAX_ENVS 1024
#define XRL_STATIC_PACK_MAX_NODES 131072
#define XRL_STATIC_PACK_MAX_EDGES 524288
xrl_status xrl_pack_csr_static(int32_t device, int32_t num_op_types, int32_t num_graphs,
                               const int32_t* n_nodes, const int32_t* n_edges, const int32_t* op,
                               const int32_t* edge_src, const int32_t* edge_dst,
                               const int32_t* env_off, int32_t num_envs, int32_t* node_off,
                               int32_t* edge_off, int32_t* seg_id, int32_t* graph_env,
                               int32_t* rowptr, int32_t* col, int32_t* device_status, void* stream);

/* Per-step timing of the path's steps with CUDA events on the launching stream (off by
 * default).  Families: 0 pack (Section 3.3.2), 1 node update (Eq. 6), 2 transform and 3
 * score/softmax/aggregate (Eq. 7), 4 readout (Eq. 8 sum), 5 global update + heads, 6 the last
 * aggregate layer when it is fused with the readout, 7 all attention layers of a small step when
 * they run as one launch (then 2, 3 and 6 stay empty).
 * xrl_profile(ctx, 1) starts recording (synchronises the device, drops earlier records);
 * xrl_profile_read synchronises the device, fills total_ms / launches (HOST,
 * [num_families]) with the time and kernel count accumulated per family since the last read,
 * and clears the records. */
xrl_status xrl_profile(xrl_ctx* ctx, int32_t enable);
xrl_status xrl_profile_read(xrl_ctx* ctx, double* total_ms, int64_t* launches, int32_t num_families);

/* Static description of the build ("sm_100a ...").  Never NULL. */
const char* xrl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* XRL_H_ */

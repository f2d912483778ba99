// CPU oracle for the X-RLflow agent's per-step forward pass.
//
// TEST INFRASTRUCTURE, NOT PRODUCT CODE.  This file is the slow, plain statement of what
// the path computes: per-node and per-edge loops in double precision, no blocking, no
// fusion, no SIMD, no BLAS.  It shares nothing with the CUDA library (no header, no
// helper, no table) and must never be called from it.  Only tests, the smoke check and
// the benchmark's CPU-baseline leg may load it.
//
// What it follows (sections and equations of the X-RLflow paper):
//   xo_pack          Section 3.3.2  the current graph and its candidates batched into one meta-graph
//   xo_encode        Section 3.4    Eq. 6 (node update), Eq. 7 (k graph-attention layers,
//                                   attention as in the GAT paper it cites), Eq. 8 (global update)
//   xo_policy_value  Section 3.3.2  two-layer MLP heads, padded action space with a boolean
//                                   mask, No-Op action; Section 3.3.3 invalid-action masking
//   xo_sample        Section 3.3.2  the action is drawn from the categorical distribution;
//                                   random words from Philox4x32-10 (Salmon et al., SC'11)
//   xo_init_weights  (no passage: the paper names no initialisation) the library's seeded Xavier-uniform blob
//   xo_ppo_grad      Section 3.3.4  Eq. 3 (clipped objective), Eq. 4 (value loss), Eq. 5 (their sum with an
//                                   entropy term) over a mini-batch, and the gradient with respect to every
//                                   weight; xo_gae: the generalised advantage estimates it is fed with
// Readings of what the paper leaves open (activation = ReLU, LeakyReLU slope 0.2 inside the
// attention score, in-neighbours plus self, heads concatenated, biases, a weight matrix in
// Eq. 8, per-graph scoring for the policy) are listed in the design notes of the repository.
//
// Parity pins: every function below is pinned by tests that do not call it to produce
// their expected values (dense-adjacency brute force in numpy, closed forms on chains and
// stars, invariants, a third-party Philox).  Nothing here is "parity unpinned".
//
// Floating point: double everywhere.  mode 0 ("exact") rounds only the inputs and those
// weights the bf16 model stores in bf16; mode 1 ("mirrored") additionally rounds Z and every
// layer output to bf16, as a debugging aid.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { XO_OK = 0, XO_INVALID_ARG = 1, XO_BAD_GRAPH = 2 };

struct Model {
  int32_t T, S, H, K, L, Hm, Dg, dtype;  // dtype: 0 fp32, 1 bf16 storage
  int32_t Hm2;                           // second hidden width of the heads' MLPs, 0 = one hidden layer
  int32_t nbr;                           // neighbourhood of Eq. 7: 0 = producers, 1 = producers and consumers
};

// bfloat16 = the upper 16 bits of an IEEE binary32; round to nearest, ties to even.
double round_bf16(double x) {
  float f = static_cast<float>(x);
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return f;  // inf / nan unchanged
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  u &= 0xFFFF0000u;
  std::memcpy(&f, &u, 4);
  return f;
}

double relu(double x) { return x > 0.0 ? x : 0.0; }
double leaky_relu(double x) { return x > 0.0 ? x : 0.2 * x; }

// Offsets into the flat weight blob (matrices row-major [in x out]).
struct Weights {
  const float* W0; const float* b0;
  std::vector<const float*> W, a_src, a_dst, b;
  const float* Wg; const float* bg;
  const float* pW1; const float* pb1; const float* pWh; const float* pbh; const float* pw2; const float* pb2;
  const float* vW1; const float* vb1; const float* vWh; const float* vbh; const float* vw2; const float* vb2;
};

Weights slice(const Model& m, const float* blob) {
  Weights w;
  const float* p = blob;
  auto take = [&](int64_t n) { const float* q = p; p += n; return q; };
  w.W0 = take(int64_t(2 * m.S + m.T) * m.H);
  w.b0 = take(m.H);
  for (int l = 0; l < m.L; ++l) {
    w.W.push_back(take(int64_t(m.H) * m.H));
    w.a_src.push_back(take(m.H));
    w.a_dst.push_back(take(m.H));
    w.b.push_back(take(m.H));
  }
  w.Wg = take(int64_t(m.H + m.Dg) * m.H);
  w.bg = take(m.H);
  // heads: Linear(in, Hm), ReLU, [Linear(Hm, Hm2), ReLU,] Linear(last hidden, 1)
  const int last = m.Hm2 > 0 ? m.Hm2 : m.Hm;
  w.pW1 = take(int64_t(m.H) * m.Hm); w.pb1 = take(m.Hm);
  w.pWh = take(int64_t(m.Hm) * m.Hm2); w.pbh = take(m.Hm2);
  w.pw2 = take(last); w.pb2 = take(1);
  w.vW1 = take(int64_t(2 * m.H) * m.Hm); w.vb1 = take(m.Hm);
  w.vWh = take(int64_t(m.Hm) * m.Hm2); w.vbh = take(m.Hm2);
  w.vw2 = take(last); w.vb2 = take(1);
  return w;
}

// A weight as the model stores it: Eq. 6 and Eq. 7 matrices live in bf16 when dtype = 1.
double stored(const Model& m, float w) { return m.dtype == 1 ? round_bf16(w) : double(w); }

// An input feature (a node's shape features, an edge's attributes) as the model stores it: the caller
// hands over arbitrary reals (Section 3.3.2: tensor shapes divided by a constant); a bf16 model keeps
// them in bf16, so they are rounded here, once, before anything is computed from them.
double stored_input(const Model& m, float v) { return m.dtype == 1 ? round_bf16(v) : double(v); }

// Encode one graph (nodes [lo, hi) of the packed batch).  Writes its H-vector to `emb`.
void encode_graph(const Model& m, const Weights& w, int32_t lo, int32_t hi,
                  const int32_t* rowptr, const int32_t* col, const int32_t* op,
                  const float* shape, const double* g_attr, int mode, double* emb,
                  int dump_layer, double* node_dump, double* alpha_edge, double* alpha_self,
                  const float* edge_attr, const int32_t* eid) {
  const int S = m.S, T = m.T, H = m.H, K = m.K, d = m.H / m.K;
  const int n = hi - lo;
  const int F0 = 2 * S + T;
  std::vector<double> h(size_t(n) * H), z(size_t(n) * H), hn(size_t(n) * H);
  std::vector<double> s_src(size_t(n) * K), s_dst(size_t(n) * K);

  auto dump = [&](int layer) {
    if (node_dump && dump_layer == layer)
      for (int i = 0; i < n; ++i)
        for (int c = 0; c < H; ++c) node_dump[size_t(lo + i) * H + c] = h[size_t(i) * H + c];
  };

  // ---- Eq. 6: h'_i = sigma( W ( sum_{j in E_i} e_j  ||  h_i ) ).
  // The attribute of edge j->i is the shape feature vector of its producer j, or, when the caller
  // gives attributes per edge (Section 3.3.2 as written: the shape of the tensor the edge carries), the
  // S values of that edge; the node attribute is the one-hot operator id followed by the node's own
  // shape features.
  std::vector<double> x(F0), W0s(size_t(F0) * H);
  for (size_t t = 0; t < W0s.size(); ++t) W0s[t] = stored(m, w.W0[t]);
  for (int i = 0; i < n; ++i) {
    const int gi = lo + i;
    for (int s = 0; s < F0; ++s) x[s] = 0.0;
    for (int e = rowptr[gi]; e < rowptr[gi + 1]; ++e)
      for (int s = 0; s < S; ++s)
        x[s] += stored_input(m, edge_attr ? edge_attr[size_t(eid[e]) * S + s] : shape[size_t(col[e]) * S + s]);
    x[S + op[gi]] = 1.0;
    for (int s = 0; s < S; ++s) x[S + T + s] = stored_input(m, shape[size_t(gi) * S + s]);
    for (int c = 0; c < H; ++c) {
      double acc = 0.0;
      for (int s = 0; s < F0; ++s) acc += x[s] * W0s[size_t(s) * H + c];
      acc += double(w.b0[c]);
      acc = relu(acc);
      h[size_t(i) * H + c] = (mode == 1 && m.dtype == 1) ? round_bf16(acc) : acc;
    }
  }
  dump(0);

  // ---- Eq. 7, k times: h'_i = sigma( sum_{j in N_i} alpha_ij W h_j ),  N_i = in(i) + {i}, or with
  // nbr = 1 the producers and the consumers of i and i itself ("neighbours of node i" read both ways);
  // repeated edges count once each, in either direction.
  std::vector<std::vector<int>> nbl(n);
  for (int i = 0; i < n; ++i)
    for (int e = rowptr[lo + i]; e < rowptr[lo + i + 1]; ++e) nbl[i].push_back(col[e] - lo);
  if (m.nbr == 1)
    for (int i = 0; i < n; ++i)      // i consumes col[e]: i is a consumer-side neighbour of that producer
      for (int e = rowptr[lo + i]; e < rowptr[lo + i + 1]; ++e) nbl[col[e] - lo].push_back(i);
  for (int l = 0; l < m.L; ++l) {
    const float* W = w.W[l];
    std::vector<double> Ws(size_t(H) * H);
    for (size_t t = 0; t < Ws.size(); ++t) Ws[t] = stored(m, W[t]);
    for (int i = 0; i < n; ++i) {   // z_i = W^T h_i, summed over the input index k in order
      for (int c = 0; c < H; ++c) z[size_t(i) * H + c] = 0.0;
      for (int k = 0; k < H; ++k)
        for (int c = 0; c < H; ++c)
          z[size_t(i) * H + c] += h[size_t(i) * H + k] * Ws[size_t(k) * H + c];
    }
    // attention half-scores per head: e_ij = LeakyReLU(a_dst . z_i + a_src . z_j), i.e. the GAT
    // score a . [z_i || z_j] with a = [a_dst || a_src], i the receiving node
    for (int i = 0; i < n; ++i)
      for (int k = 0; k < K; ++k) {
        double ss = 0.0, sd = 0.0;
        for (int c = 0; c < d; ++c) {
          ss += double(w.a_src[l][k * d + c]) * z[size_t(i) * H + k * d + c];
          sd += double(w.a_dst[l][k * d + c]) * z[size_t(i) * H + k * d + c];
        }
        s_src[size_t(i) * K + k] = ss;
        s_dst[size_t(i) * K + k] = sd;
      }
    if (mode == 1 && m.dtype == 1)
      for (auto& v : z) v = round_bf16(v);

    for (int i = 0; i < n; ++i) {
      const int gi = lo + i;
      const int e0 = rowptr[gi], e1 = rowptr[gi + 1];
      const int din = e1 - e0;                          // the first din neighbours are the producers
      const int deg = int(nbl[i].size());
      std::vector<double> sc(deg + 1), al(deg + 1);
      for (int k = 0; k < K; ++k) {
        double mx = -INFINITY;
        for (int t = 0; t <= deg; ++t) {
          const int j = (t < deg) ? nbl[i][t] : i;   // last entry is the self term
          sc[t] = leaky_relu(s_src[size_t(j) * K + k] + s_dst[size_t(i) * K + k]);
          if (sc[t] > mx) mx = sc[t];
        }
        double sum = 0.0;
        for (int t = 0; t <= deg; ++t) { al[t] = std::exp(sc[t] - mx); sum += al[t]; }
        for (int t = 0; t <= deg; ++t) al[t] /= sum;
        if (dump_layer == l + 1 && alpha_edge) {
          for (int t = 0; t < din; ++t) alpha_edge[size_t(e0 + t) * K + k] = al[t];
          alpha_self[size_t(gi) * K + k] = al[deg];
        }
        for (int c = k * d; c < (k + 1) * d; ++c) {
          double acc = 0.0;
          for (int t = 0; t <= deg; ++t) {
            const int j = (t < deg) ? nbl[i][t] : i;
            acc += al[t] * z[size_t(j) * H + c];
          }
          acc = relu(acc + double(w.b[l][c]));
          hn[size_t(i) * H + c] = (mode == 1 && m.dtype == 1) ? round_bf16(acc) : acc;
        }
      }
    }
    h.swap(hn);
    dump(l + 1);
  }

  // ---- Eq. 8: g' = sigma( W_g ( sum_N h  ||  g ) + b_g )
  std::vector<double> u(H + m.Dg, 0.0);
  for (int i = 0; i < n; ++i)
    for (int c = 0; c < H; ++c) u[c] += h[size_t(i) * H + c];
  for (int c = 0; c < m.Dg; ++c) u[H + c] = g_attr ? g_attr[c] : 0.0;
  for (int c = 0; c < H; ++c) {
    double acc = 0.0;
    for (int k = 0; k < H + m.Dg; ++k) acc += u[k] * double(w.Wg[size_t(k) * H + c]);
    emb[c] = relu(acc + double(w.bg[c]));
  }
}

// The heads' MLP (Section 3.3.2: "two layers"; the hyper-parameter table lists hidden sizes [256, 64]):
// y1 = ReLU(W1^T x + b1); with a second hidden width, y2 = ReLU(Wh^T y1 + bh); out = w2 . y_last + b2.
double mlp_scalar(const double* x, int in, int hid, int hid2, const float* W1, const float* b1,
                  const float* Wh, const float* bh, const float* w2, const float* b2) {
  std::vector<double> y1(hid);
  for (int c = 0; c < hid; ++c) {
    double acc = double(b1[c]);
    for (int k = 0; k < in; ++k) acc += x[k] * double(W1[size_t(k) * hid + c]);
    y1[c] = relu(acc);
  }
  double out = double(b2[0]);
  if (hid2 <= 0) {
    for (int c = 0; c < hid; ++c) out += y1[c] * double(w2[c]);
    return out;
  }
  for (int c = 0; c < hid2; ++c) {
    double acc = double(bh[c]);
    for (int k = 0; k < hid; ++k) acc += y1[k] * double(Wh[size_t(k) * hid2 + c]);
    out += relu(acc) * double(w2[c]);
  }
  return out;
}

// ---- Section 3.3.4: the PPO objective of one mini-batch (Eq. 3, 4, 5) and its gradient ---------------
// A mini-batch is a packed batch whose environments are stored transitions: environment e holds the state
// (current graph + candidates), the action that was taken there, the old policy's log-probability of it,
// its advantage estimate and its value target.
//   ratio_e = pi(a_e | s_e) / pi_old(a_e | s_e)
//   L_clip  = - mean_e min(ratio_e A_e, clip(ratio_e, 1 - eps, 1 + eps) A_e)          (Eq. 3)
//   L_vf    =   mean_e (V(s_e) - R_e)^2                                                (Eq. 4)
//   L_ent   =   mean_e sum_a pi(a | s_e) log pi(a | s_e)        (minus the entropy, over the valid actions)
//   J       =   L_clip + c1 L_vf + c2 L_ent                                            (Eq. 5)
// The gradient is taken by hand, layer by layer in reverse, with respect to every entry of the weight blob
// (for a bf16 model: with respect to the stored, rounded values).  ReLU'(0) = 0, LeakyReLU'(0) = 0.2, and
// the derivative of the clipped objective is that of whichever term of the min is the smaller one.
// mode 1 ("mirrored", a debugging aid like xo_encode's): the forward pass keeps Z and every layer's output
// rounded to bf16, as a bf16 model stores them, and the reverse pass runs at those values with the rounding
// treated as the identity; mode 2 is mode 1 with the half-scores taken from the rounded Z instead of the
// exact one (the two places an implementation may take them from).  mode 0 is the definition.

// Forward intermediates of one graph that the reverse pass needs.
struct GraphTape {
  int n = 0;
  std::vector<std::vector<int>> nbl;                 // neighbours of each node (self excluded)
  std::vector<double> x0;                            // [n x F0] inputs of Eq. 6
  std::vector<std::vector<double>> h;                // h[l]: [n x H] after Eq. 6 (l = 0) and after layer l
  std::vector<std::vector<double>> z, s_src, s_dst;  // per layer: [n x H], [n x K], [n x K]
  std::vector<std::vector<double>> alpha;            // per layer: for node i, head k: deg_i + 1 weights, packed
  std::vector<size_t> aoff;                          // start of node i's weights inside alpha[l] (times K)
  std::vector<double> u, emb;                        // Eq. 8 input [H + Dg] and output [H]
};

void forward_tape(const Model& m, const Weights& w, int32_t lo, int32_t hi, const int32_t* rowptr,
                  const int32_t* col, const int32_t* op, const float* shape, const double* g_attr,
                  const float* edge_attr, const int32_t* eid, int mode, GraphTape& tp) {
  const int S = m.S, T = m.T, H = m.H, K = m.K, d = m.H / m.K, F0 = 2 * S + T;
  const int n = hi - lo;
  const bool mirror = (mode != 0 && m.dtype == 1);   // keep Z and the layer outputs as a bf16 model stores them
  tp.n = n;
  tp.nbl.assign(n, {});
  for (int i = 0; i < n; ++i)
    for (int e = rowptr[lo + i]; e < rowptr[lo + i + 1]; ++e) tp.nbl[i].push_back(col[e] - lo);
  if (m.nbr == 1)
    for (int i = 0; i < n; ++i)
      for (int e = rowptr[lo + i]; e < rowptr[lo + i + 1]; ++e) tp.nbl[col[e] - lo].push_back(i);
  tp.aoff.assign(n + 1, 0);
  for (int i = 0; i < n; ++i) tp.aoff[i + 1] = tp.aoff[i] + tp.nbl[i].size() + 1;
  tp.x0.assign(size_t(n) * F0, 0.0);
  tp.h.assign(m.L + 1, std::vector<double>(size_t(n) * H));
  tp.z.assign(m.L, std::vector<double>(size_t(n) * H));
  tp.s_src.assign(m.L, std::vector<double>(size_t(n) * K));
  tp.s_dst.assign(m.L, std::vector<double>(size_t(n) * K));
  tp.alpha.assign(m.L, std::vector<double>(tp.aoff[n] * K));
  // Eq. 6
  for (int i = 0; i < n; ++i) {
    const int gi = lo + i;
    double* x = &tp.x0[size_t(i) * F0];
    for (int e = rowptr[gi]; e < rowptr[gi + 1]; ++e)
      for (int s = 0; s < S; ++s)
        x[s] += stored_input(m, edge_attr ? edge_attr[size_t(eid[e]) * S + s] : shape[size_t(col[e]) * S + s]);
    x[S + op[gi]] = 1.0;
    for (int s = 0; s < S; ++s) x[S + T + s] = stored_input(m, shape[size_t(gi) * S + s]);
    for (int c = 0; c < H; ++c) {
      double acc = double(w.b0[c]);
      for (int s = 0; s < F0; ++s) acc += x[s] * stored(m, w.W0[size_t(s) * H + c]);
      tp.h[0][size_t(i) * H + c] = mirror ? round_bf16(relu(acc)) : relu(acc);
    }
  }
  // Eq. 7
  for (int l = 0; l < m.L; ++l) {
    const std::vector<double>& hin = tp.h[l];
    std::vector<double>& z = tp.z[l];
    for (int i = 0; i < n; ++i)
      for (int c = 0; c < H; ++c) {
        double acc = 0.0;
        for (int k = 0; k < H; ++k) acc += hin[size_t(i) * H + k] * stored(m, w.W[l][size_t(k) * H + c]);
        z[size_t(i) * H + c] = (mirror && mode == 2) ? round_bf16(acc) : acc;
      }
    for (int i = 0; i < n; ++i)
      for (int k = 0; k < K; ++k) {
        double ss = 0.0, sd = 0.0;
        for (int c = 0; c < d; ++c) {
          ss += double(w.a_src[l][k * d + c]) * z[size_t(i) * H + k * d + c];
          sd += double(w.a_dst[l][k * d + c]) * z[size_t(i) * H + k * d + c];
        }
        tp.s_src[l][size_t(i) * K + k] = ss;
        tp.s_dst[l][size_t(i) * K + k] = sd;
      }
    if (mirror)
      for (auto& v : z) v = round_bf16(v);
    for (int i = 0; i < n; ++i) {
      const int deg = int(tp.nbl[i].size());
      for (int k = 0; k < K; ++k) {
        double* al = &tp.alpha[l][(tp.aoff[i]) * K + size_t(k) * (deg + 1)];
        double mx = -INFINITY;
        for (int t = 0; t <= deg; ++t) {
          const int j = (t < deg) ? tp.nbl[i][t] : i;
          al[t] = leaky_relu(tp.s_src[l][size_t(j) * K + k] + tp.s_dst[l][size_t(i) * K + k]);
          if (al[t] > mx) mx = al[t];
        }
        double sum = 0.0;
        for (int t = 0; t <= deg; ++t) { al[t] = std::exp(al[t] - mx); sum += al[t]; }
        for (int t = 0; t <= deg; ++t) al[t] /= sum;
        for (int c = k * d; c < (k + 1) * d; ++c) {
          double acc = 0.0;
          for (int t = 0; t <= deg; ++t) acc += al[t] * z[size_t((t < deg) ? tp.nbl[i][t] : i) * H + c];
          const double out = relu(acc + double(w.b[l][c]));
          tp.h[l + 1][size_t(i) * H + c] = mirror ? round_bf16(out) : out;
        }
      }
    }
  }
  // Eq. 8
  tp.u.assign(H + m.Dg, 0.0);
  tp.emb.assign(H, 0.0);
  for (int i = 0; i < n; ++i)
    for (int c = 0; c < H; ++c) tp.u[c] += tp.h[m.L][size_t(i) * H + c];
  for (int c = 0; c < m.Dg; ++c) tp.u[H + c] = g_attr ? g_attr[c] : 0.0;
  for (int c = 0; c < H; ++c) {
    double acc = double(w.bg[c]);
    for (int k = 0; k < H + m.Dg; ++k) acc += tp.u[k] * double(w.Wg[size_t(k) * H + c]);
    tp.emb[c] = relu(acc);
  }
}

// Reverse pass of one graph: demb = dJ / d emb of this graph; adds into the blob-shaped gradient `g`
// (pointers of `gw` address it the way `w` addresses the weights).
struct GradPtrs {
  double* W0; double* b0;
  std::vector<double*> W, a_src, a_dst, b;
  double* Wg; double* bg;
  double *pW1, *pb1, *pWh, *pbh, *pw2, *pb2, *vW1, *vb1, *vWh, *vbh, *vw2, *vb2;
};

void backward_graph(const Model& m, const Weights& w, const GraphTape& tp, const double* demb, GradPtrs& gw) {
  const int S = m.S, T = m.T, H = m.H, K = m.K, d = m.H / m.K, F0 = 2 * S + T, n = tp.n;
  // Eq. 8
  std::vector<double> dpre(H), du(H + m.Dg, 0.0);
  for (int c = 0; c < H; ++c) dpre[c] = tp.emb[c] > 0.0 ? demb[c] : 0.0;
  for (int k = 0; k < H + m.Dg; ++k)
    for (int c = 0; c < H; ++c) {
      gw.Wg[size_t(k) * H + c] += tp.u[k] * dpre[c];
      du[k] += double(w.Wg[size_t(k) * H + c]) * dpre[c];
    }
  for (int c = 0; c < H; ++c) gw.bg[c] += dpre[c];
  std::vector<double> dh(size_t(n) * H), dz(size_t(n) * H), dhin(size_t(n) * H);
  for (int i = 0; i < n; ++i)
    for (int c = 0; c < H; ++c) dh[size_t(i) * H + c] = du[c];      // the readout is a plain sum
  // Eq. 7, last layer first
  for (int l = m.L - 1; l >= 0; --l) {
    const std::vector<double>& hout = tp.h[l + 1];
    const std::vector<double>& hin = tp.h[l];
    const std::vector<double>& z = tp.z[l];
    std::vector<double> ds_src(size_t(n) * K, 0.0), ds_dst(size_t(n) * K, 0.0);
    std::fill(dz.begin(), dz.end(), 0.0);
    for (int i = 0; i < n; ++i) {
      const int deg = int(tp.nbl[i].size());
      std::vector<double> dal(deg + 1);
      for (int k = 0; k < K; ++k) {
        const double* al = &tp.alpha[l][(tp.aoff[i]) * K + size_t(k) * (deg + 1)];
        // through ReLU and the bias
        double dp[512];
        for (int c = 0; c < d; ++c) {
          const int cc = k * d + c;
          dp[c] = hout[size_t(i) * H + cc] > 0.0 ? dh[size_t(i) * H + cc] : 0.0;
          gw.b[l][cc] += dp[c];
        }
        // out = sum_t al[t] z_{j_t}: to the weights and to the gathered rows
        for (int t = 0; t <= deg; ++t) {
          const int j = (t < deg) ? tp.nbl[i][t] : i;
          double acc = 0.0;
          for (int c = 0; c < d; ++c) {
            acc += dp[c] * z[size_t(j) * H + k * d + c];
            dz[size_t(j) * H + k * d + c] += al[t] * dp[c];
          }
          dal[t] = acc;
        }
        // softmax, then LeakyReLU, then the sum of the two half-scores
        double dot = 0.0;
        for (int t = 0; t <= deg; ++t) dot += al[t] * dal[t];
        for (int t = 0; t <= deg; ++t) {
          const int j = (t < deg) ? tp.nbl[i][t] : i;
          const double e = tp.s_src[l][size_t(j) * K + k] + tp.s_dst[l][size_t(i) * K + k];
          const double de = al[t] * (dal[t] - dot) * (e > 0.0 ? 1.0 : 0.2);
          ds_src[size_t(j) * K + k] += de;
          ds_dst[size_t(i) * K + k] += de;
        }
      }
    }
    // half-scores are dot products of z with the attention vectors
    for (int i = 0; i < n; ++i)
      for (int k = 0; k < K; ++k)
        for (int c = 0; c < d; ++c) {
          const int cc = k * d + c;
          const double zs = z[size_t(i) * H + cc];
          gw.a_src[l][cc] += ds_src[size_t(i) * K + k] * zs;
          gw.a_dst[l][cc] += ds_dst[size_t(i) * K + k] * zs;
          dz[size_t(i) * H + cc] += ds_src[size_t(i) * K + k] * double(w.a_src[l][cc]) +
                                    ds_dst[size_t(i) * K + k] * double(w.a_dst[l][cc]);
        }
    // z = h W
    for (int i = 0; i < n; ++i)
      for (int k = 0; k < H; ++k) {
        double acc = 0.0;
        for (int c = 0; c < H; ++c) {
          gw.W[l][size_t(k) * H + c] += hin[size_t(i) * H + k] * dz[size_t(i) * H + c];
          acc += stored(m, w.W[l][size_t(k) * H + c]) * dz[size_t(i) * H + c];
        }
        dhin[size_t(i) * H + k] = acc;
      }
    dh.swap(dhin);
  }
  // Eq. 6
  for (int i = 0; i < n; ++i)
    for (int c = 0; c < H; ++c) {
      const double dp = tp.h[0][size_t(i) * H + c] > 0.0 ? dh[size_t(i) * H + c] : 0.0;
      gw.b0[c] += dp;
      for (int s = 0; s < F0; ++s) gw.W0[size_t(s) * H + c] += tp.x0[size_t(i) * F0 + s] * dp;
    }
}

// A head's MLP forward keeping its hidden activations, and its reverse pass given d out.
struct MlpTape { std::vector<double> y1, y2; };
double mlp_forward_tape(const double* x, int in, int hid, int hid2, const float* W1, const float* b1,
                        const float* Wh, const float* bh, const float* w2, const float* b2, MlpTape& tp) {
  tp.y1.assign(hid, 0.0);
  tp.y2.assign(hid2 > 0 ? hid2 : 0, 0.0);
  for (int c = 0; c < hid; ++c) {
    double acc = double(b1[c]);
    for (int k = 0; k < in; ++k) acc += x[k] * double(W1[size_t(k) * hid + c]);
    tp.y1[c] = relu(acc);
  }
  double out = double(b2[0]);
  if (hid2 <= 0) {
    for (int c = 0; c < hid; ++c) out += tp.y1[c] * double(w2[c]);
    return out;
  }
  for (int c = 0; c < hid2; ++c) {
    double acc = double(bh[c]);
    for (int k = 0; k < hid; ++k) acc += tp.y1[k] * double(Wh[size_t(k) * hid2 + c]);
    tp.y2[c] = relu(acc);
    out += tp.y2[c] * double(w2[c]);
  }
  return out;
}
void mlp_backward(const double* x, int in, int hid, int hid2, const float* W1, const float* Wh, const float* w2,
                  const MlpTape& tp, double dout, double* gW1, double* gb1, double* gWh, double* gbh,
                  double* gw2, double* gb2, double* dx) {
  gb2[0] += dout;
  std::vector<double> dy1(hid, 0.0);
  if (hid2 <= 0) {
    for (int c = 0; c < hid; ++c) {
      gw2[c] += tp.y1[c] * dout;
      dy1[c] = tp.y1[c] > 0.0 ? double(w2[c]) * dout : 0.0;
    }
  } else {
    for (int c = 0; c < hid2; ++c) {
      gw2[c] += tp.y2[c] * dout;
      const double da = tp.y2[c] > 0.0 ? double(w2[c]) * dout : 0.0;
      gbh[c] += da;
      for (int k = 0; k < hid; ++k) {
        gWh[size_t(k) * hid2 + c] += tp.y1[k] * da;
        dy1[k] += double(Wh[size_t(k) * hid2 + c]) * da;
      }
    }
    for (int k = 0; k < hid; ++k)
      if (!(tp.y1[k] > 0.0)) dy1[k] = 0.0;
  }
  for (int c = 0; c < hid; ++c) gb1[c] += dy1[c];
  for (int k = 0; k < in; ++k) {
    double acc = 0.0;
    for (int c = 0; c < hid; ++c) {
      gW1[size_t(k) * hid + c] += x[k] * dy1[c];
      acc += double(W1[size_t(k) * hid + c]) * dy1[c];
    }
    if (dx) dx[k] += acc;
  }
}

inline void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
  uint64_t p = uint64_t(a) * uint64_t(b);
  hi = uint32_t(p >> 32);
  lo = uint32_t(p);
}

}  // namespace

extern "C" {

// Philox4x32 with 10 rounds, from its published definition (Salmon, Moraes, Dror, Shaw,
// "Parallel random numbers: as easy as 1, 2, 3", SC'11): round = two 32x32->64 multiplies,
// a word permutation and a key xor; the key is bumped by the Weyl constants between rounds.
void xo_philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1, uint32_t c2,
                      uint32_t c3, uint32_t* out) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo(M0, c0, hi0, lo0);
    mulhilo(M1, c2, hi1, lo1);
    uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Section 3.3.2: batch the B graphs into one meta-graph.  CSR by destination over global
// node ids; inside a row the sources keep the order of the input edge list.
int xo_pack(int32_t B, const int32_t* n_nodes, const int32_t* n_edges, const int32_t* edge_src,
            const int32_t* edge_dst, int32_t num_envs, const int32_t* env_off,
            int32_t* node_off, int32_t* edge_off, int32_t* seg_id, int32_t* graph_env,
            int32_t* rowptr, int32_t* col, int32_t* eid) {
  // eid (optional, [E]): the input edge that ends up in each CSR slot, for attributes that live on edges
  if (B < 0 || num_envs < 0) return XO_INVALID_ARG;
  node_off[0] = 0; edge_off[0] = 0;
  for (int g = 0; g < B; ++g) {
    if (n_nodes[g] < 0 || n_edges[g] < 0) return XO_INVALID_ARG;
    node_off[g + 1] = node_off[g] + n_nodes[g];
    edge_off[g + 1] = edge_off[g] + n_edges[g];
  }
  if (env_off[0] != 0 || env_off[num_envs] != B) return XO_INVALID_ARG;
  for (int e = 0; e < num_envs; ++e) {
    if (env_off[e + 1] <= env_off[e]) return XO_INVALID_ARG;  // each env has its current graph
    for (int g = env_off[e]; g < env_off[e + 1]; ++g) graph_env[g] = e;
  }
  const int32_t N = node_off[B];
  for (int g = 0; g < B; ++g)
    for (int i = node_off[g]; i < node_off[g + 1]; ++i) seg_id[i] = g;
  for (int i = 0; i <= N; ++i) rowptr[i] = 0;
  for (int g = 0; g < B; ++g)
    for (int e = edge_off[g]; e < edge_off[g + 1]; ++e) {
      const int32_t s = edge_src[e], t = edge_dst[e];
      if (s < 0 || s >= n_nodes[g] || t < 0 || t >= n_nodes[g] || s == t) return XO_BAD_GRAPH;
      rowptr[node_off[g] + t + 1] += 1;
    }
  for (int i = 0; i < N; ++i) rowptr[i + 1] += rowptr[i];
  std::vector<int32_t> cursor(rowptr, rowptr + N);
  for (int g = 0; g < B; ++g)
    for (int e = edge_off[g]; e < edge_off[g + 1]; ++e) {
      const int32_t t = node_off[g] + edge_dst[e];
      if (eid) eid[cursor[t]] = e;
      col[cursor[t]++] = node_off[g] + edge_src[e];
    }
  return XO_OK;
}

// Section 3.4: Eq. 6 -> L x Eq. 7 -> Eq. 8 for the graphs listed in `sel` (all when null).
// graph_emb is [n_sel x H].  node_dump (optional, [N x H]) receives the node features after
// stage `dump_layer` (0 = Eq. 6, l = l-th attention layer) for the selected graphs;
// alpha_edge [E x K] / alpha_self [N x K] (optional) receive that layer's attention weights.
int xo_encode(const Model* m, const float* weights, int32_t B, const int32_t* node_off,
              const int32_t* rowptr, const int32_t* col, const int32_t* op, const float* shape,
              const double* g0, int32_t n_sel, const int32_t* sel, int32_t mode,
              int32_t threads, double* graph_emb, int32_t dump_layer, double* node_dump,
              double* alpha_edge, double* alpha_self, const float* edge_attr, const int32_t* eid) {
  // edge_attr (optional, [E x S], input edge order) with eid from xo_pack: attributes on edges in Eq. 6
  if (m->H % m->K != 0 || m->L < 0) return XO_INVALID_ARG;
  if (edge_attr && !eid) return XO_INVALID_ARG;
  const Weights w = slice(*m, weights);
  const int count = sel ? n_sel : B;
  int bad = 0;
#ifdef _OPENMP
  if (threads > 0) omp_set_num_threads(threads);
#pragma omp parallel for schedule(dynamic, 1)
#endif
  for (int t = 0; t < count; ++t) {
    const int g = sel ? sel[t] : t;
    if (g < 0 || g >= B) { bad = 1; continue; }
    encode_graph(*m, w, node_off[g], node_off[g + 1], rowptr, col, op, shape,
                 g0 ? g0 + size_t(g) * m->Dg : nullptr, mode, graph_emb + size_t(t) * m->H,
                 dump_layer, node_dump, alpha_edge, alpha_self, edge_attr, eid);
  }
  (void)threads;
  return bad ? XO_INVALID_ARG : XO_OK;
}

// Section 3.3.2 / 3.3.3: policy and value heads over the graph embeddings of each
// environment.  graph env_off[e] is the current graph, the following ones its candidates.
// logits/probs are [num_envs x (A_max+1)], the last column is No-Op (scored by the current
// graph).  Invalid and padded actions get probability exactly 0 (logit reported as -inf).
int xo_policy_value(const Model* m, const float* weights, int32_t num_envs,
                    const int32_t* env_off, int32_t A_max, const double* graph_emb,
                    const uint8_t* mask, double* logits, double* probs, double* value) {
  const Weights w = slice(*m, weights);
  const int H = m->H, A1 = A_max + 1;
  for (int e = 0; e < num_envs; ++e) {
    const int cur = env_off[e];
    const int C = env_off[e + 1] - env_off[e] - 1;
    if (C < 0 || C > A_max) return XO_INVALID_ARG;
    for (int a = C; a < A_max; ++a)
      if (mask[size_t(e) * A_max + a]) return XO_INVALID_ARG;
    double* lg = logits + size_t(e) * A1;
    double* pr = probs + size_t(e) * A1;
    double mx = -INFINITY;
    for (int a = 0; a < A1; ++a) {
      const bool valid = (a == A_max) || mask[size_t(e) * A_max + a];
      const int g = (a == A_max) ? cur : cur + 1 + a;
      lg[a] = valid ? mlp_scalar(graph_emb + size_t(g) * H, H, m->Hm, m->Hm2, w.pW1, w.pb1, w.pWh, w.pbh, w.pw2, w.pb2)
                    : -INFINITY;
      if (lg[a] > mx) mx = lg[a];
    }
    double sum = 0.0;
    for (int a = 0; a < A1; ++a) {
      pr[a] = (lg[a] == -INFINITY) ? 0.0 : std::exp(lg[a] - mx);
      sum += pr[a];
    }
    for (int a = 0; a < A1; ++a) pr[a] /= sum;

    // value: MLP over [ current graph || mean of the valid candidates ]
    std::vector<double> u(2 * H, 0.0);
    int nv = 0;
    for (int c = 0; c < H; ++c) u[c] = graph_emb[size_t(cur) * H + c];
    for (int a = 0; a < C; ++a)
      if (mask[size_t(e) * A_max + a]) {
        ++nv;
        for (int c = 0; c < H; ++c) u[H + c] += graph_emb[size_t(cur + 1 + a) * H + c];
      }
    if (nv > 0)
      for (int c = 0; c < H; ++c) u[H + c] /= double(nv);
    value[e] = mlp_scalar(u.data(), 2 * H, m->Hm, m->Hm2, w.vW1, w.vb1, w.vWh, w.vbh, w.vw2, w.vb2);
  }
  return XO_OK;
}

// Draw one action per environment from fp32 probabilities with integer arithmetic only.
// q_a = floor(p_a * 2^32); Q = sum q_a; r = 64 random bits from Philox keyed by the seed with
// counter (env, step lo, step hi, 0); t = floor(r * Q / 2^64); the action is the first index
// whose inclusive prefix sum of q exceeds t.  Q = 0 yields No-Op (the last index).
int xo_sample(int32_t num_envs, int32_t A1, const float* probs, uint64_t seed, uint64_t step,
              int32_t* action) {
  for (int e = 0; e < num_envs; ++e) {
    uint32_t r[4];
    xo_philox4x32_10(uint32_t(seed), uint32_t(seed >> 32), uint32_t(e), uint32_t(step),
                     uint32_t(step >> 32), 0u, r);
    const uint64_t r64 = uint64_t(r[0]) | (uint64_t(r[1]) << 32);
    uint64_t Q = 0;
    for (int a = 0; a < A1; ++a) {
      const float p = probs[size_t(e) * A1 + a];
      if (!(p >= 0.0f) || p > 1.0f) return XO_INVALID_ARG;
      Q += uint64_t(std::floor(double(p) * 4294967296.0));
    }
    int32_t act = A1 - 1;
    if (Q > 0) {
      const uint64_t t = uint64_t((static_cast<unsigned __int128>(r64) * Q) >> 64);
      uint64_t run = 0;
      for (int a = 0; a < A1; ++a) {
        run += uint64_t(std::floor(double(probs[size_t(e) * A1 + a]) * 4294967296.0));
        if (run > t) { act = a; break; }
      }
    }
    action[e] = act;
  }
  return XO_OK;
}

// Eq. 3-5 over the environments of a packed batch and the gradient of J with respect to the weight blob.
// action [num_envs] in [0, A_max] (A_max = No-Op) must be a valid action of its environment; logp_old, adv,
// ret [num_envs]; loss_out[4] = {J, L_clip, L_vf, L_ent}; grad = blob-shaped, double; logp_out (optional,
// [num_envs]) receives log pi(a_e | s_e) of the current weights.
int xo_ppo_grad(const Model* m, const float* weights, int32_t B, const int32_t* node_off,
                const int32_t* rowptr, const int32_t* col, const int32_t* op, const float* shape,
                const double* g0, const float* edge_attr, const int32_t* eid, int32_t num_envs,
                const int32_t* env_off, int32_t A_max, const uint8_t* mask, const int32_t* action,
                const double* logp_old, const double* adv, const double* ret, double eps, double c1,
                double c2, double* loss_out, double* grad, double* logp_out, int32_t mode) {
  if (m->H % m->K != 0 || m->L < 0 || num_envs <= 0 || m->H / m->K > 512) return XO_INVALID_ARG;
  if (edge_attr && !eid) return XO_INVALID_ARG;
  const Weights w = slice(*m, weights);
  const int H = m->H;
  // gradient pointers laid out like the blob
  GradPtrs gw;
  {
    double* p = grad;
    auto take = [&](int64_t nn) { double* q = p; p += nn; return q; };
    const int last = m->Hm2 > 0 ? m->Hm2 : m->Hm;
    gw.W0 = take(int64_t(2 * m->S + m->T) * H); gw.b0 = take(H);
    for (int l = 0; l < m->L; ++l) {
      gw.W.push_back(take(int64_t(H) * H)); gw.a_src.push_back(take(H));
      gw.a_dst.push_back(take(H)); gw.b.push_back(take(H));
    }
    gw.Wg = take(int64_t(H + m->Dg) * H); gw.bg = take(H);
    gw.pW1 = take(int64_t(H) * m->Hm); gw.pb1 = take(m->Hm);
    gw.pWh = take(int64_t(m->Hm) * m->Hm2); gw.pbh = take(m->Hm2);
    gw.pw2 = take(last); gw.pb2 = take(1);
    gw.vW1 = take(int64_t(2 * H) * m->Hm); gw.vb1 = take(m->Hm);
    gw.vWh = take(int64_t(m->Hm) * m->Hm2); gw.vbh = take(m->Hm2);
    gw.vw2 = take(last); gw.vb2 = take(1);
    for (double* q = grad; q < p; ++q) *q = 0.0;
  }
  // forward of every graph, kept
  std::vector<GraphTape> tapes(B);
  for (int g = 0; g < B; ++g)
    forward_tape(*m, w, node_off[g], node_off[g + 1], rowptr, col, op, shape,
                 g0 ? g0 + size_t(g) * m->Dg : nullptr, edge_attr, eid, mode, tapes[g]);
  std::vector<double> demb(size_t(B) * H, 0.0);
  double Lclip = 0.0, Lvf = 0.0, Lent = 0.0;
  const double inv_ne = 1.0 / double(num_envs);
  for (int e = 0; e < num_envs; ++e) {
    const int cur = env_off[e];
    const int C = env_off[e + 1] - cur - 1;
    if (C < 0 || C > A_max) return XO_INVALID_ARG;
    const int A1 = A_max + 1;
    // policy logits of the valid actions, their MLP tapes
    std::vector<double> lg(A1, -INFINITY), pr(A1, 0.0);
    std::vector<MlpTape> mt(A1);
    double mx = -INFINITY;
    for (int a = 0; a < A1; ++a) {
      const bool valid = (a == A_max) || (a < C && mask[size_t(e) * A_max + a]);
      if (a < A_max && a >= C && mask[size_t(e) * A_max + a]) return XO_INVALID_ARG;
      if (!valid) continue;
      const int g = (a == A_max) ? cur : cur + 1 + a;
      lg[a] = mlp_forward_tape(tapes[g].emb.data(), H, m->Hm, m->Hm2, w.pW1, w.pb1, w.pWh, w.pbh, w.pw2,
                               w.pb2, mt[a]);
      if (lg[a] > mx) mx = lg[a];
    }
    double sum = 0.0;
    for (int a = 0; a < A1; ++a)
      if (lg[a] != -INFINITY) { pr[a] = std::exp(lg[a] - mx); sum += pr[a]; }
    for (int a = 0; a < A1; ++a) pr[a] /= sum;
    const int act = action[e];
    if (act < 0 || act > A_max || lg[act] == -INFINITY) return XO_INVALID_ARG;
    const double logp = (lg[act] - mx) - std::log(sum);
    if (logp_out) logp_out[e] = logp;
    // Eq. 3
    const double ratio = std::exp(logp - logp_old[e]);
    const double clipped = ratio < 1.0 - eps ? 1.0 - eps : (ratio > 1.0 + eps ? 1.0 + eps : ratio);
    const double t1 = ratio * adv[e], t2 = clipped * adv[e];
    Lclip += -(t1 <= t2 ? t1 : t2) * inv_ne;
    const double dlogp = (t1 <= t2) ? -adv[e] * ratio * inv_ne : 0.0;   // the clipped term is flat where it is active
    // entropy term
    double plogp = 0.0;
    for (int a = 0; a < A1; ++a)
      if (pr[a] > 0.0) plogp += pr[a] * std::log(pr[a]);
    Lent += plogp * inv_ne;
    // d J / d logit_b = dlogp (1[b = act] - p_b) + c2 / Ne * p_b (log p_b - sum_a p_a log p_a)
    for (int a = 0; a < A1; ++a) {
      if (lg[a] == -INFINITY) continue;
      double dl = dlogp * ((a == act ? 1.0 : 0.0) - pr[a]);
      if (pr[a] > 0.0) dl += c2 * inv_ne * pr[a] * (std::log(pr[a]) - plogp);
      const int g = (a == A_max) ? cur : cur + 1 + a;
      mlp_backward(tapes[g].emb.data(), H, m->Hm, m->Hm2, w.pW1, w.pWh, w.pw2, mt[a], dl, gw.pW1, gw.pb1,
                   gw.pWh, gw.pbh, gw.pw2, gw.pb2, &demb[size_t(g) * H]);
    }
    // Eq. 4: value head over [ current graph || mean of the valid candidates ]
    std::vector<double> u(2 * H, 0.0), du(2 * H, 0.0);
    int nv = 0;
    for (int c = 0; c < H; ++c) u[c] = tapes[cur].emb[c];
    for (int a = 0; a < C; ++a)
      if (mask[size_t(e) * A_max + a]) {
        ++nv;
        for (int c = 0; c < H; ++c) u[H + c] += tapes[cur + 1 + a].emb[c];
      }
    if (nv > 0)
      for (int c = 0; c < H; ++c) u[H + c] /= double(nv);
    MlpTape vt;
    const double v = mlp_forward_tape(u.data(), 2 * H, m->Hm, m->Hm2, w.vW1, w.vb1, w.vWh, w.vbh, w.vw2,
                                      w.vb2, vt);
    Lvf += (v - ret[e]) * (v - ret[e]) * inv_ne;
    mlp_backward(u.data(), 2 * H, m->Hm, m->Hm2, w.vW1, w.vWh, w.vw2, vt, c1 * 2.0 * (v - ret[e]) * inv_ne,
                 gw.vW1, gw.vb1, gw.vWh, gw.vbh, gw.vw2, gw.vb2, du.data());
    for (int c = 0; c < H; ++c) demb[size_t(cur) * H + c] += du[c];
    if (nv > 0)
      for (int a = 0; a < C; ++a)
        if (mask[size_t(e) * A_max + a])
          for (int c = 0; c < H; ++c) demb[size_t(cur + 1 + a) * H + c] += du[H + c] / double(nv);
  }
  for (int g = 0; g < B; ++g) backward_graph(*m, w, tapes[g], &demb[size_t(g) * H], gw);
  loss_out[0] = Lclip + c1 * Lvf + c2 * Lent;
  loss_out[1] = Lclip; loss_out[2] = Lvf; loss_out[3] = Lent;
  return XO_OK;
}

// Generalised advantage estimation over one trajectory of T steps (the estimator the paper takes its
// advantages from): delta_t = r_t + gamma V_{t+1} (1 - done_t) - V_t,
// A_t = delta_t + gamma lambda (1 - done_t) A_{t+1}; value targets R_t = A_t + V_t.  values has T + 1 entries
// (the last one bootstraps the tail).
int xo_gae(int32_t T, const double* reward, const double* values, const uint8_t* done, double gamma,
           double lambda, double* adv, double* ret) {
  if (T < 0) return XO_INVALID_ARG;
  double run = 0.0;
  for (int t = T - 1; t >= 0; --t) {
    const double nd = done[t] ? 0.0 : 1.0;
    const double delta = reward[t] + gamma * values[t + 1] * nd - values[t];
    run = delta + gamma * lambda * nd * run;
    adv[t] = run;
    ret[t] = run + values[t];
  }
  return XO_OK;
}

// Seeded initial weights (the paper names no initialisation; Xavier-uniform is the library's documented choice):
// matrices U(-b, b) with b = sqrt(6 / (fan_in + fan_out)), attention vectors with fan (H / K, 1), the heads' last
// layers with fan (hidden, 1), biases U(-0.1, 0.1), in blob order.  Element i is b * u_i with
// u_i = (w >> 8) 2^-23 - 1, w = first word of Philox4x32-10(key = seed, counter = (i, 0, 0, 1)).
// `out` holds the whole blob; returns the number of elements written.
int64_t xo_init_weights(const Model* m, uint64_t seed, float* out) {
  const int64_t S = m->S, T = m->T, H = m->H, Hm = m->Hm, Hm2 = m->Hm2, Dg = m->Dg, d = m->H / m->K;
  const int64_t last = Hm2 > 0 ? Hm2 : Hm;
  int64_t off = 0;
  auto xavier = [](int64_t fan_in, int64_t fan_out) { return float(std::sqrt(6.0 / double(fan_in + fan_out))); };
  auto fill = [&](int64_t count, float bound) {
    for (int64_t t = 0; t < count; ++t) {
      const uint64_t i = uint64_t(off + t);
      uint32_t w[4];
      xo_philox4x32_10(uint32_t(seed), uint32_t(seed >> 32), uint32_t(i), uint32_t(i >> 32), 0u, 1u, w);
      const float u = float(w[0] >> 8) * 1.1920928955078125e-07f - 1.0f;    // both steps are exact in float
      out[off + t] = bound * u;
    }
    off += count;
  };
  const float bias = 0.1f;
  fill((2 * S + T) * H, xavier(2 * S + T, H)); fill(H, bias);
  for (int l = 0; l < m->L; ++l) {
    fill(H * H, xavier(H, H));
    fill(H, xavier(d, 1)); fill(H, xavier(d, 1));
    fill(H, bias);
  }
  fill((H + Dg) * H, xavier(H + Dg, H)); fill(H, bias);
  for (int head = 0; head < 2; ++head) {
    const int64_t in = head == 0 ? H : 2 * H;
    fill(in * Hm, xavier(in, Hm)); fill(Hm, bias);
    if (Hm2 > 0) { fill(Hm * Hm2, xavier(Hm, Hm2)); fill(Hm2, bias); }
    fill(last, xavier(last, 1)); fill(1, bias);
  }
  return off;
}

int xo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"

// CPU oracle for the VARCO partitioned graph-convolution layer.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
// the paper's method computes; the CUDA library is checked against it.  It is
// never part of the product path: nothing but the tests, the smoke check and
// the benchmark's CPU-baseline leg may load it.  It shares no code, header,
// table or helper with the CUDA library.
//
// What it follows (paper: "Distributed Training of Large Graph Neural Networks
// with Variable Communication Rates"):
//   * layer math                      -- Eq. (2) with K = 2 taps, i.e. one AGGREGATE
//                                        per layer (Section II), SAGE convolution and
//                                        ReLU (Section V)
//   * who computes what, what is sent -- Section III, Section III-A, Algorithm 1
//   * compress / decompress           -- Definition 1 and the appendix
//                                        "Compression Mechanism": send F/c values of a
//                                        row, positions random and known to the decoder
//                                        through a shared key, zeros elsewhere
//   * backward through the compressor -- Algorithm 1 (back-propagate across machines
//                                        through the compression routine), Section III-A
//   * scheduler                       -- Section IV and the appendix "Scheduler" (linear ratio schedule
//                                        of the experiments; fixed-increment, linear and exponential
//                                        rate schedules; fixed ratios and "no communication" of Section V)
//
// All floating point is fp64.  Loops are written in the order of the
// algorithm's steps; there is no blocking or fusion.  OpenMP is used only on
// loops whose iterations write disjoint outputs.
//
// Pins (see tests): full communication == centralized layer; dense-matrix
// brute force on <= 10 nodes incl. autograd gradients; finite differences;
// mask / byte-count invariants; schedule closed forms; keyed-permutation test
// vectors.  Parity unpinned: nothing in this file -- accuracy curves and
// convergence are not computed here at all.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------- shared random key
// The paper only says that encoder and decoder share a random key generator
// (appendix "Compression Mechanism").  The concrete generator is this
// library's own definition: a 6-round balanced Feistel network over the
// smallest even-bit domain covering [0, F), cycle-walked into [0, F), keyed by
// (seed, epoch, layer, global node id) through a 64-bit mixer.
const uint64_t PHI64 = 0x9E3779B97F4A7C15ull;  // floor(2^64 / golden ratio)
const uint64_t A64 = 0x6A09E667F3BCC909ull;    // frac(sqrt 2) * 2^64, forced odd
const uint64_t B64 = 0xBB67AE8584CAA73Bull;    // frac(sqrt 3) * 2^64, forced odd
const uint32_t G32 = 0x9E3779B9u;              // floor(2^32 / golden ratio)

uint64_t mix64(uint64_t x) {
  x ^= x >> 32;
  x *= A64;
  x ^= x >> 29;
  x *= B64;
  x ^= x >> 32;
  return x;
}

struct KeyedPerm {
  uint32_t rk[6];
  int h;
  uint32_t msk;
  uint32_t F;

  KeyedPerm(uint64_t seed, uint32_t epoch, uint32_t layer, uint64_t node, int width) {
    uint64_t a = mix64(seed ^ PHI64);
    a = mix64(a + epoch);
    a = mix64(a + layer);
    a = mix64(a + node);
    for (int i = 0; i < 6; ++i) rk[i] = (uint32_t)(mix64(a + (uint64_t)(i + 1) * PHI64) >> 32);
    F = (uint32_t)width;
    int bits = 0;
    while (((uint64_t)1 << bits) < (uint64_t)width) ++bits;  // bitlen(F-1) for F >= 2
    if (bits < 2) bits = 2;
    if (bits & 1) ++bits;
    h = bits / 2;
    msk = ((uint32_t)1 << h) - 1u;
  }
  uint32_t f(int i, uint32_t r) const { return (uint32_t)((r + rk[i]) * G32) >> (32 - h); }
  uint32_t enc(uint32_t x) const {
    uint32_t L = x >> h, R = x & msk;
    for (int i = 0; i < 6; ++i) {
      uint32_t t = L ^ f(i, R);
      L = R;
      R = t;
    }
    return (L << h) | R;
  }
  uint32_t dec(uint32_t y) const {
    uint32_t L = y >> h, R = y & msk;
    for (int i = 5; i >= 0; --i) {
      uint32_t t = R ^ f(i, L);
      R = L;
      L = t;
    }
    return (L << h) | R;
  }
  uint32_t pi(uint32_t m) const {
    uint32_t x = enc(m);
    while (x >= F) x = enc(x);
    return x;
  }
  uint32_t pi_inv(uint32_t c) const {
    uint32_t x = dec(c);
    while (x >= F) x = dec(x);
    return x;
  }
};

// ---------------------------------------------------------------- rate -> kept elements
// Definition 1 sends F / c values; c is kept as the exact rational num/den.
// Reading for non-integer F/c: k = ceil(F / c) clamped to [1, F].
// den == 0 stands for the "no communication" setting of Section V (Tables II-III): an unbounded
// ratio, nothing is sent, k = 0, and every remote row is the all-zero vector at the receiver.
int kept_elements(int F, uint64_t num, uint64_t den) {
  if (F <= 0 || num == 0) return -1;
  if (den == 0) return 0;
  if (num < den) return -1;
  uint64_t k = ((uint64_t)F * den + num - 1) / num;
  if (k < 1) k = 1;
  if (k > (uint64_t)F) k = (uint64_t)F;
  return (int)k;
}

// ---------------------------------------------------------------- graph + partition
struct Graph {
  int64_t n = 0;
  int P = 0;
  int conv = 0;  // 0 = GCN (self-loop, symmetric normalisation), 1 = SAGE-mean
  std::vector<int64_t> rp;
  std::vector<int32_t> col;
  std::vector<int32_t> part;
  // halo[p * P + q] = ascending global ids of the nodes owned by p that some
  // node of q aggregates from (Section III: "the nodes in the boundary").
  std::vector<std::vector<int64_t>> halo;
  std::vector<int64_t> new_to_old;  // partition-contiguous order, ascending id inside a part
  int64_t H_total = 0, cross = 0, self_ = 0;
  // transpose (who aggregates from j), built on demand
  std::vector<int64_t> trp;
  std::vector<int32_t> tcol;

  double weight(int64_t i, int64_t j) const {
    // entry s_ij of the aggregation matrix, degrees taken from the whole graph
    double di = (double)(rp[i + 1] - rp[i]);
    if (conv == 1) return di > 0 ? 1.0 / di : 0.0;
    double dj = (double)(rp[j + 1] - rp[j]);
    return 1.0 / std::sqrt((di + 1.0) * (dj + 1.0));
  }
  void build_transpose() {
    if (!trp.empty()) return;
    trp.assign(n + 1, 0);
    for (int64_t e = 0; e < rp[n]; ++e) trp[col[e] + 1]++;
    for (int64_t i = 0; i < n; ++i) trp[i + 1] += trp[i];
    tcol.resize(rp[n]);
    std::vector<int64_t> fill(trp.begin(), trp.end() - 1);
    for (int64_t i = 0; i < n; ++i)
      for (int64_t e = rp[i]; e < rp[i + 1]; ++e) tcol[fill[col[e]]++] = (int32_t)i;
  }
};

struct LayerArgs {
  int F_in, F_out, relu;
  const double *X, *W_self, *W_neigh, *bias;
  uint64_t num, den;
  uint64_t seed;
  uint32_t epoch, layer;
  int elem_bytes;
};

// Position of the m-th value on the wire.  For k < F the kept positions are the first k images of
// the keyed permutation, sent in that order.  At full communication (k == F) nothing is dropped
// and the row is sent as it is: the paper's "full communication" setting involves no compressor,
// and the order of a complete row on the wire is not observable in its terms.
uint32_t wire_position(const KeyedPerm& kp, int m, int k) {
  return (k == (int)kp.F) ? (uint32_t)m : kp.pi((uint32_t)m);
}
// compress one row: z[m] = x[position(m)], m < k   (appendix "Compression Mechanism")
void compress_row(const KeyedPerm& kp, const double* x, int k, double* z) {
  for (int m = 0; m < k; ++m) z[m] = x[wire_position(kp, m, k)];
}
// decompress one row: values put back in place, zero everywhere else
void decompress_row(const KeyedPerm& kp, const double* z, int k, int F, double* xt) {
  for (int c = 0; c < F; ++c) xt[c] = 0.0;
  for (int m = 0; m < k; ++m) xt[wire_position(kp, m, k)] = z[m];
}

// Steps 2-3 of Algorithm 1 for one layer: every worker p compresses its
// boundary rows for every adjacent worker q and "sends" them; q decompresses.
// xt holds the decompressed rows in q's receive order (q, then p, then id).
// Returns the number of values that crossed a partition boundary.
uint64_t exchange_forward(const Graph& g, const LayerArgs& a, int k, std::vector<double>& xt,
                          std::vector<int64_t>& slot_base /* P*P */) {
  const int F = a.F_in;
  xt.assign((size_t)g.H_total * F, 0.0);
  slot_base.assign((size_t)g.P * g.P, 0);
  int64_t s = 0;
  for (int q = 0; q < g.P; ++q)
    for (int p = 0; p < g.P; ++p) {
      slot_base[(size_t)p * g.P + q] = s;
      s += (int64_t)g.halo[(size_t)p * g.P + q].size();
    }
  uint64_t sent = 0;
  std::vector<double> z(F);
  for (int p = 0; p < g.P; ++p)
    for (int q = 0; q < g.P; ++q) {
      const std::vector<int64_t>& rows = g.halo[(size_t)p * g.P + q];
      for (size_t r = 0; r < rows.size(); ++r) {
        int64_t j = rows[r];
        KeyedPerm kp(a.seed, a.epoch, a.layer, (uint64_t)j, F);
        compress_row(kp, a.X + j * F, k, z.data());       // at the owner p
        sent += (uint64_t)k;                               // k values on the wire
        decompress_row(kp, z.data(), k, F, &xt[(size_t)(slot_base[(size_t)p * g.P + q] + (int64_t)r) * F]);  // at q
      }
    }
  return sent;
}

// slot_of[j] for the receiving worker q (or -1): where q keeps its copy of row j
void fill_slot_lookup(const Graph& g, int q, const std::vector<int64_t>& slot_base, std::vector<int64_t>& slot_of) {
  std::fill(slot_of.begin(), slot_of.end(), (int64_t)-1);
  for (int p = 0; p < g.P; ++p) {
    const std::vector<int64_t>& rows = g.halo[(size_t)p * g.P + q];
    for (size_t r = 0; r < rows.size(); ++r) slot_of[rows[r]] = slot_base[(size_t)p * g.P + q] + (int64_t)r;
  }
}

// Step 3 of Algorithm 1: aggregate with exact local rows and decompressed remote rows.
void aggregate(const Graph& g, const LayerArgs& a, const std::vector<double>& xt,
               const std::vector<int64_t>& slot_base, double* agg) {
  const int F = a.F_in;
  std::vector<int64_t> slot_of(g.n);
  for (int q = 0; q < g.P; ++q) {
    fill_slot_lookup(g, q, slot_base, slot_of);
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < g.n; ++i) {
      if (g.part[i] != q) continue;
      double* out = agg + i * F;
      for (int c = 0; c < F; ++c) out[c] = 0.0;
      if (g.conv == 0) {  // GCN self-loop: always local, exact
        double w = g.weight(i, i);
        for (int c = 0; c < F; ++c) out[c] += w * a.X[i * F + c];
      }
      for (int64_t e = g.rp[i]; e < g.rp[i + 1]; ++e) {
        int64_t j = g.col[e];
        double w = g.weight(i, j);
        const double* u = (g.part[j] == q) ? a.X + j * F : &xt[(size_t)slot_of[j] * F];
        for (int c = 0; c < F; ++c) out[c] += w * u[c];
      }
    }
  }
}

// Eq. (2): pre-activation of row i.  SAGE: x_i W_self + agg_i W_neigh + b;  GCN: agg_i W + b.
void transform_row(const Graph& g, const LayerArgs& a, const double* xi, const double* aggi, double* z) {
  for (int o = 0; o < a.F_out; ++o) z[o] = a.bias ? a.bias[o] : 0.0;
  for (int c = 0; c < a.F_in; ++c) {
    double v = aggi[c];
    const double* w = a.W_neigh + (size_t)c * a.F_out;
    for (int o = 0; o < a.F_out; ++o) z[o] += v * w[o];
  }
  if (g.conv == 1)
    for (int c = 0; c < a.F_in; ++c) {
      double v = xi[c];
      const double* w = a.W_self + (size_t)c * a.F_out;
      for (int o = 0; o < a.F_out; ++o) z[o] += v * w[o];
    }
}

}  // namespace

extern "C" {

void orc_set_threads(int t) {
#ifdef _OPENMP
  if (t > 0) omp_set_num_threads(t);
#else
  (void)t;
#endif
}
int orc_get_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

uint64_t orc_mix64(uint64_t x) { return mix64(x); }

void orc_round_keys(uint64_t seed, uint32_t epoch, uint32_t layer, uint64_t node, int F, uint32_t* rk6) {
  KeyedPerm kp(seed, epoch, layer, node, F);
  for (int i = 0; i < 6; ++i) rk6[i] = kp.rk[i];
}

// idx[m] = pi(m), m < k: the positions of the k values that are sent
int orc_perm_indices(uint64_t seed, uint32_t epoch, uint32_t layer, uint64_t node, int F, int k, int32_t* idx) {
  if (F < 1 || k < 0 || k > F) return -1;
  KeyedPerm kp(seed, epoch, layer, node, F);
  for (int m = 0; m < k; ++m) idx[m] = (int32_t)kp.pi((uint32_t)m);
  return 0;
}
// positions of the k values of a row in the order they are sent
int orc_wire_positions(uint64_t seed, uint32_t epoch, uint32_t layer, uint64_t node, int F, int k, int32_t* idx) {
  if (F < 1 || k < 0 || k > F) return -1;
  KeyedPerm kp(seed, epoch, layer, node, F);
  for (int m = 0; m < k; ++m) idx[m] = (int32_t)wire_position(kp, m, k);
  return 0;
}
int orc_perm_inverse(uint64_t seed, uint32_t epoch, uint32_t layer, uint64_t node, int F, int c) {
  KeyedPerm kp(seed, epoch, layer, node, F);
  return (int)kp.pi_inv((uint32_t)c);
}

int orc_kept(int F, uint64_t num, uint64_t den) { return kept_elements(F, num, den); }

// Linear scheduler of the appendix "Scheduler", with the clip read as a lower
// clip at c_min:  c_e = max(c_max - a (c_max - c_min) e / K, c_min), kept as the
// exact rational num/den with den = K.
int orc_schedule_linear(int epoch, int K, int a, int c_max, int c_min, uint64_t* num, uint64_t* den) {
  if (K <= 0 || a <= 0 || c_min < 1 || c_max < c_min || epoch < 0) return -1;
  int64_t v = (int64_t)c_max * K - (int64_t)a * (c_max - c_min) * (int64_t)epoch;
  if (v < (int64_t)c_min * K) v = (int64_t)c_min * K;
  *num = (uint64_t)v;
  *den = (uint64_t)K;
  return 0;
}

// The other schedulers of the appendix "Scheduler".  There r_k is the communicated FRACTION (the
// "compress rate", increasing while training); the ratio handed to the compressor is c_k = 1 / r_k.
// Fractions are kept as integers over a common denominator, clipped at 1 (full communication).
//
// Fixed increment, written as the recurrence it is stated as: r_0 = r0/den, r_{k+1} = r_k + R/den.
int orc_schedule_fixed_increment(int epoch, uint64_t r0, uint64_t R, uint64_t den, uint64_t* num_out,
                                 uint64_t* den_out) {
  if (epoch < 0 || den == 0 || r0 == 0 || r0 > den) return -1;
  uint64_t r = r0;
  for (int e = 0; e < epoch; ++e) {
    r += R;
    if (r > den) r = den;
  }
  *num_out = den;   // c = 1 / (r / den) = den / r
  *den_out = r;
  return 0;
}
// Linear increase in closed form: r_k = alpha k + r_0 with alpha = alpha_num/den, r_0 = r0/den.
int orc_schedule_rate_linear(int epoch, uint64_t r0, uint64_t alpha_num, uint64_t den, uint64_t* num_out,
                             uint64_t* den_out) {
  if (epoch < 0 || den == 0 || r0 == 0 || r0 > den) return -1;
  // alpha k + r_0 >= 1 as soon as k >= (den - r0) / alpha_num: clip there without forming the product
  uint64_t r = den;
  if (alpha_num == 0) r = r0;
  else if ((uint64_t)epoch <= (den - r0) / alpha_num) r = r0 + alpha_num * (uint64_t)epoch;
  if (r > den) r = den;
  *num_out = den;
  *den_out = r;
  return 0;
}
// Exponential increase r_k = 1 / beta^(K - k + 1), k = 1..K; epoch e = k - 1, so c_e = beta^(K - e):
// the last epoch e = K - 1 still compresses by beta (full communication would be step K + 1).
// The power saturates at 2^32 - 1 (any ratio above the row width keeps one element).
int orc_schedule_exponential(int epoch, int K, int beta, uint64_t* num_out, uint64_t* den_out) {
  if (epoch < 0 || K < 1 || beta < 2) return -1;
  uint64_t c = 1;
  for (int i = 0; i < K - epoch; ++i) {
    c *= (uint64_t)beta;
    if (c > 0xFFFFFFFFull) {
      c = 0xFFFFFFFFull;
      break;
    }
  }
  *num_out = c;
  *den_out = 1;
  return 0;
}

// ------------------------------------------------------------ graph handle
void* orc_graph_create(int64_t n, const int64_t* rp, const int32_t* col, const int32_t* part, int P, int conv) {
  Graph* g = new Graph;
  g->n = n;
  g->P = P;
  g->conv = conv;
  g->rp.assign(rp, rp + n + 1);
  g->col.assign(col, col + rp[n]);
  g->part.assign(part, part + n);
  g->halo.assign((size_t)P * P, std::vector<int64_t>());
  // boundary sets: j in V_p is in halo(p -> q) iff some i in V_q has an entry (i, j)
  std::vector<char> seen(n);
  for (int q = 0; q < P; ++q) {
    std::fill(seen.begin(), seen.end(), 0);
    for (int64_t i = 0; i < n; ++i) {
      if (part[i] != q) continue;
      for (int64_t e = rp[i]; e < rp[i + 1]; ++e) {
        int64_t j = col[e];
        if (part[j] != q) seen[j] = 1;
      }
    }
    for (int64_t j = 0; j < n; ++j)
      if (seen[j]) g->halo[(size_t)part[j] * P + q].push_back(j);
  }
  for (int64_t i = 0; i < n; ++i)
    for (int64_t e = rp[i]; e < rp[i + 1]; ++e) {
      if (part[col[e]] != part[i]) g->cross++;
      else g->self_++;
    }
  for (size_t s = 0; s < g->halo.size(); ++s) g->H_total += (int64_t)g->halo[s].size();
  for (int p = 0; p < P; ++p)
    for (int64_t i = 0; i < n; ++i)
      if (part[i] == p) g->new_to_old.push_back(i);
  return g;
}
void orc_graph_destroy(void* h) { delete (Graph*)h; }
int64_t orc_graph_H_total(void* h) { return ((Graph*)h)->H_total; }
int64_t orc_graph_cross_entries(void* h) { return ((Graph*)h)->cross; }
int64_t orc_graph_self_entries(void* h) { return ((Graph*)h)->self_; }
void orc_graph_counts(void* h, int64_t* PxP) {
  Graph* g = (Graph*)h;
  for (size_t s = 0; s < g->halo.size(); ++s) PxP[s] = (int64_t)g->halo[s].size();
}
void orc_graph_halo(void* h, int p, int q, int64_t* out) {
  Graph* g = (Graph*)h;
  const std::vector<int64_t>& v = g->halo[(size_t)p * g->P + q];
  std::copy(v.begin(), v.end(), out);
}
void orc_graph_perm(void* h, int64_t* new_to_old) {
  Graph* g = (Graph*)h;
  std::copy(g->new_to_old.begin(), g->new_to_old.end(), new_to_old);
}

// ------------------------------------------------------------ compress / decompress over the plan
// packed: rows in send order (owner p, destination q, ascending id), k values each.
int orc_compress(void* h, const double* X, int F, uint64_t num, uint64_t den, uint64_t seed, uint32_t epoch,
                 uint32_t layer, double* packed, uint64_t* values_sent) {
  Graph* g = (Graph*)h;
  int k = kept_elements(F, num, den);
  if (k < 0) return -1;
  size_t pos = 0;
  for (int p = 0; p < g->P; ++p)
    for (int q = 0; q < g->P; ++q)
      for (int64_t j : g->halo[(size_t)p * g->P + q]) {
        KeyedPerm kp(seed, epoch, layer, (uint64_t)j, F);
        compress_row(kp, X + j * F, k, packed + pos * k);
        ++pos;
      }
  if (values_sent) *values_sent = (uint64_t)pos * (uint64_t)k;
  return 0;
}
// Xhalo: rows in receive order (destination q, owner p, ascending id), F values each.
int orc_decompress(void* h, const double* packed, int F, uint64_t num, uint64_t den, uint64_t seed, uint32_t epoch,
                   uint32_t layer, double* Xhalo) {
  Graph* g = (Graph*)h;
  int k = kept_elements(F, num, den);
  if (k < 0) return -1;
  // send-order base of every (p, q) segment
  std::vector<int64_t> send_base((size_t)g->P * g->P);
  int64_t s = 0;
  for (int p = 0; p < g->P; ++p)
    for (int q = 0; q < g->P; ++q) {
      send_base[(size_t)p * g->P + q] = s;
      s += (int64_t)g->halo[(size_t)p * g->P + q].size();
    }
  int64_t slot = 0;
  for (int q = 0; q < g->P; ++q)
    for (int p = 0; p < g->P; ++p) {
      const std::vector<int64_t>& rows = g->halo[(size_t)p * g->P + q];
      for (size_t r = 0; r < rows.size(); ++r) {
        KeyedPerm kp(seed, epoch, layer, (uint64_t)rows[r], F);
        decompress_row(kp, packed + (size_t)(send_base[(size_t)p * g->P + q] + (int64_t)r) * k, k, F,
                       Xhalo + (size_t)slot * F);
        ++slot;
      }
    }
  return 0;
}

// ------------------------------------------------------------ layer forward (all partitions)
// X [n x F_in], Y [n x F_out], Agg [n x F_in] in ORIGINAL node order.
int orc_layer_fwd(void* h, int F_in, int F_out, int relu, const double* X, const double* W_self,
                  const double* W_neigh, const double* bias, uint64_t num, uint64_t den, uint64_t seed,
                  uint32_t epoch, uint32_t layer, int elem_bytes, double* Y, double* Agg, uint64_t* halo_bytes) {
  Graph* g = (Graph*)h;
  LayerArgs a{F_in, F_out, relu, X, W_self, W_neigh, bias, num, den, seed, epoch, layer, elem_bytes};
  int k = kept_elements(F_in, num, den);
  if (k < 0) return -1;
  if (g->conv == 1 && !W_self) return -1;
  std::vector<double> xt;
  std::vector<int64_t> slot_base;
  uint64_t sent = exchange_forward(*g, a, k, xt, slot_base);
  std::vector<double> agg_local;
  double* agg = Agg;
  if (!agg) {
    agg_local.resize((size_t)g->n * F_in);
    agg = agg_local.data();
  }
  aggregate(*g, a, xt, slot_base, agg);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < g->n; ++i) {
    std::vector<double> z(F_out);
    transform_row(*g, a, X + i * F_in, agg + i * F_in, z.data());
    for (int o = 0; o < F_out; ++o) Y[i * F_out + o] = (relu && z[o] < 0.0) ? 0.0 : z[o];
  }
  if (halo_bytes) *halo_bytes = sent * (uint64_t)elem_bytes;
  return 0;
}

// ------------------------------------------------------------ layer backward (all partitions)
// Given dY and the forward output Y (the ReLU mask is 1[Y > 0]).
// dW_self, dW_neigh, dbias are sums over the nodes of ALL partitions (third
// communication round of Section III-A).  The halo-row gradients are compressed
// with the SAME key and k as the forward pass and returned to the owner.
int orc_layer_bwd(void* h, int F_in, int F_out, int relu, const double* X, const double* Y, const double* W_self,
                  const double* W_neigh, const double* dY, uint64_t num, uint64_t den, uint64_t seed,
                  uint32_t epoch, uint32_t layer, int elem_bytes, double* dX, double* dW_self, double* dW_neigh,
                  double* dbias, uint64_t* halo_bytes) {
  Graph* g = (Graph*)h;
  LayerArgs a{F_in, F_out, relu, X, W_self, W_neigh, nullptr, num, den, seed, epoch, layer, elem_bytes};
  int k = kept_elements(F_in, num, den);
  if (k < 0) return -1;
  const int64_t n = g->n;
  // forward pieces needed by the weight gradient: agg
  std::vector<double> xt;
  std::vector<int64_t> slot_base;
  exchange_forward(*g, a, k, xt, slot_base);
  std::vector<double> agg((size_t)n * F_in);
  aggregate(*g, a, xt, slot_base, agg.data());

  std::vector<double> dZ((size_t)n * F_out), dagg((size_t)n * F_in);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    for (int o = 0; o < F_out; ++o)
      dZ[i * F_out + o] = (relu && !(Y[i * F_out + o] > 0.0)) ? 0.0 : dY[i * F_out + o];
    for (int c = 0; c < F_in; ++c) {
      double s = 0.0, t = 0.0;
      for (int o = 0; o < F_out; ++o) {
        s += dZ[i * F_out + o] * W_neigh[(size_t)c * F_out + o];
        if (g->conv == 1) t += dZ[i * F_out + o] * W_self[(size_t)c * F_out + o];
      }
      dagg[i * F_in + c] = s;
      dX[i * F_in + c] = (g->conv == 1) ? t : 0.0;
    }
  }
  // weight gradients: summed over every node of every partition
  for (int c = 0; c < F_in * F_out; ++c) {
    dW_neigh[c] = 0.0;
    if (g->conv == 1) dW_self[c] = 0.0;
  }
  for (int o = 0; o < F_out; ++o) dbias[o] = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    for (int o = 0; o < F_out; ++o) dbias[o] += dZ[i * F_out + o];
    for (int c = 0; c < F_in; ++c) {
      double av = agg[i * F_in + c], xv = X[i * F_in + c];
      for (int o = 0; o < F_out; ++o) {
        dW_neigh[(size_t)c * F_out + o] += av * dZ[i * F_out + o];
        if (g->conv == 1) dW_self[(size_t)c * F_out + o] += xv * dZ[i * F_out + o];
      }
    }
  }
  // back through the aggregation: each worker q pushes gradients to its local
  // rows directly and to its halo slots; the halo-slot gradients are then
  // compressed, returned to the owner and added there.
  std::vector<double> ghalo((size_t)g->H_total * F_in, 0.0);
  std::vector<int64_t> slot_of(n);
  for (int q = 0; q < g->P; ++q) {
    fill_slot_lookup(*g, q, slot_base, slot_of);
    for (int64_t i = 0; i < n; ++i) {
      if (g->part[i] != q) continue;
      const double* di = &dagg[i * F_in];
      if (g->conv == 0) {
        double w = g->weight(i, i);
        for (int c = 0; c < F_in; ++c) dX[i * F_in + c] += w * di[c];
      }
      for (int64_t e = g->rp[i]; e < g->rp[i + 1]; ++e) {
        int64_t j = g->col[e];
        double w = g->weight(i, j);
        double* dst = (g->part[j] == q) ? dX + j * F_in : &ghalo[(size_t)slot_of[j] * F_in];
        for (int c = 0; c < F_in; ++c) dst[c] += w * di[c];
      }
    }
  }
  uint64_t sent = 0;
  std::vector<double> z(F_in), back(F_in);
  for (int q = 0; q < g->P; ++q)
    for (int p = 0; p < g->P; ++p) {
      const std::vector<int64_t>& rows = g->halo[(size_t)p * g->P + q];
      for (size_t r = 0; r < rows.size(); ++r) {
        int64_t j = rows[r];
        KeyedPerm kp(seed, epoch, layer, (uint64_t)j, F_in);
        compress_row(kp, &ghalo[(size_t)(slot_base[(size_t)p * g->P + q] + (int64_t)r) * F_in], k, z.data());  // at q
        sent += (uint64_t)k;
        decompress_row(kp, z.data(), k, F_in, back.data());                                                      // at p
        for (int c = 0; c < F_in; ++c) dX[j * F_in + c] += back[c];
      }
    }
  if (halo_bytes) *halo_bytes = sent * (uint64_t)elem_bytes;
  return 0;
}

// ------------------------------------------------------------ single rows, straight from the definitions
// Output row i of the layer without building any halo table: remote neighbours
// enter as M_j (.) x_j with M_j the 0/1 mask of the kept positions of row j.
// Used to check sampled outputs on graphs too large for the full tables.
int orc_layer_fwd_rows(void* h, int F_in, int F_out, int relu, const double* X, const double* W_self,
                       const double* W_neigh, const double* bias, uint64_t num, uint64_t den, uint64_t seed,
                       uint32_t epoch, uint32_t layer, const int64_t* rows, int64_t nrows, double* Y_rows,
                       double* Agg_rows) {
  Graph* g = (Graph*)h;
  LayerArgs a{F_in, F_out, relu, X, W_self, W_neigh, bias, num, den, seed, epoch, layer, 0};
  int k = kept_elements(F_in, num, den);
  if (k < 0) return -1;
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t r = 0; r < nrows; ++r) {
    int64_t i = rows[r];
    std::vector<double> agg(F_in, 0.0), z(F_out);
    if (g->conv == 0) {
      double w = g->weight(i, i);
      for (int c = 0; c < F_in; ++c) agg[c] += w * X[i * F_in + c];
    }
    for (int64_t e = g->rp[i]; e < g->rp[i + 1]; ++e) {
      int64_t j = g->col[e];
      double w = g->weight(i, j);
      if (g->part[j] == g->part[i]) {
        for (int c = 0; c < F_in; ++c) agg[c] += w * X[j * F_in + c];
      } else {
        KeyedPerm kp(seed, epoch, layer, (uint64_t)j, F_in);
        for (int m = 0; m < k; ++m) {
          uint32_t c = kp.pi((uint32_t)m);
          agg[c] += w * X[j * F_in + c];
        }
      }
    }
    transform_row(*g, a, X + i * F_in, agg.data(), z.data());
    for (int o = 0; o < F_out; ++o) Y_rows[r * F_out + o] = (relu && z[o] < 0.0) ? 0.0 : z[o];
    if (Agg_rows)
      for (int c = 0; c < F_in; ++c) Agg_rows[r * F_in + c] = agg[c];
  }
  return 0;
}

// Input-gradient row j straight from the definition:
//   dx_j = [SAGE] dZ_j W_self^T + sum_{i : j in N(i)} s_ij (part(i) == part(j) ? 1 : M_j) (.) (dZ_i W_neigh^T)
int orc_layer_dx_rows(void* h, int F_in, int F_out, int relu, const double* Y, const double* W_self,
                      const double* W_neigh, const double* dY, uint64_t num, uint64_t den, uint64_t seed,
                      uint32_t epoch, uint32_t layer, const int64_t* rows, int64_t nrows, double* dX_rows) {
  Graph* g = (Graph*)h;
  int k = kept_elements(F_in, num, den);
  if (k < 0) return -1;
  g->build_transpose();
#pragma omp parallel for schedule(dynamic, 4)
  for (int64_t r = 0; r < nrows; ++r) {
    int64_t j = rows[r];
    std::vector<double> out(F_in, 0.0), remote(F_in, 0.0), dz(F_out);
    auto masked_dz = [&](int64_t i) {
      for (int o = 0; o < F_out; ++o) dz[o] = (relu && !(Y[i * F_out + o] > 0.0)) ? 0.0 : dY[i * F_out + o];
    };
    masked_dz(j);
    if (g->conv == 1)
      for (int c = 0; c < F_in; ++c) {
        double t = 0.0;
        for (int o = 0; o < F_out; ++o) t += dz[o] * W_self[(size_t)c * F_out + o];
        out[c] += t;
      }
    if (g->conv == 0) {
      double w = g->weight(j, j);
      for (int c = 0; c < F_in; ++c) {
        double t = 0.0;
        for (int o = 0; o < F_out; ++o) t += dz[o] * W_neigh[(size_t)c * F_out + o];
        out[c] += w * t;
      }
    }
    for (int64_t e = g->trp[j]; e < g->trp[j + 1]; ++e) {
      int64_t i = g->tcol[e];
      double w = g->weight(i, j);
      masked_dz(i);
      double* dst = (g->part[i] == g->part[j]) ? out.data() : remote.data();
      for (int c = 0; c < F_in; ++c) {
        double t = 0.0;
        for (int o = 0; o < F_out; ++o) t += dz[o] * W_neigh[(size_t)c * F_out + o];
        dst[c] += w * t;
      }
    }
    KeyedPerm kp(seed, epoch, layer, (uint64_t)j, F_in);
    for (int m = 0; m < k; ++m) {
      uint32_t c = kp.pi((uint32_t)m);
      out[c] += remote[c];
    }
    for (int c = 0; c < F_in; ++c) dX_rows[r * F_in + c] = out[c];
  }
  return 0;
}

}  // extern "C"

// CPU oracle for the importance-weighted-pruning step.   TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct statement of what one data-parallel step of the
// paper's method computes for W simulated workers, written from the paper's
// Algorithm 1 and Section 3.2.  It shares no code, header, table or constant with
// the CUDA library and must never be linked, imported or called by it; only the
// tests, the smoke check and the benchmark's CPU-baseline leg may use it.
//
// Where the selection has a plain definition (the k best elements of a layer under
// a total order) the oracle is that definition: order the layer by (importance
// descending, index ascending) with a library partial-ordering routine and keep the
// first k.  There is no radix select, no histogram, no blocking or fusion here.
//
// Arithmetic: IEEE-754 binary32, round to nearest even, one operation at a time
// (build with -ffp-contract=off, never -ffast-math), denormals kept.
//
// Readings of points the paper leaves open (the same readings bind the CUDA path):
//   * Algorithm 1's first update line is the residual accumulator G += grad, and the
//     importance is taken on the accumulated value (Section 3.2: the residual is
//     accumulated locally).
//   * importance = |G| / (|w| + eps), eps > 0, instead of the unguarded |G / w|.
//   * the threshold of Algorithm 1 is the k-th largest importance of the worker's
//     layer, k = ceil(n / ratio) clamped to [1, n]; ties keep the lower index.
//   * one randomly chosen node per step supplies the index set (Section 3.2); optionally several chosen
//     nodes r_1..r_n, drawn without replacement, whose index sets are OR-ed (Algorithm 1: Mask = OR Mask_ri),
//     or one chosen node per LAYER (Algorithm 1 draws the node inside its loop over layers).
//   * Eq. 3's momentum acts on the locally kept residual: G <- m * G + grad (two roundings);
//     m = 1, the default, is the plain accumulation of Section 3.2.
//   * threshold mode is Algorithm 1 as printed: only the chosen node forms a mask, per layer
//     Mask = importance > thr[layer] (strict), the index set has whatever size results, and no
//     other worker makes a selection of its own.
//   * Section 3.3's random gradient selection (threshold mode, optional): an element whose importance
//     does not exceed the threshold is sent iff u < importance / thr, u one 24-bit uniform draw per
//     element and step, the quotient in fp32.
//   * Section 3.4's layer-wise threshold (threshold mode, optional; Eq. 4 with its two branches read as
//     "v > C" and "otherwise"): per chosen node and layer, thr = alpha + beta v if v > C else alpha - beta v,
//     v = var / mean of the layer's importances on that node.  So that the value does not depend on a
//     summation order, S1 = sum imp and S2 = sum imp^2 are the EXACT sums, each rounded once to binary64;
//     then, one binary64 operation at a time, mean = S1 / n, var = S2 / n - mean * mean (population
//     variance), v = var / mean (0 if mean = 0), thr rounded to binary32, -0 taken as +0.
//   * the ring all-reduce is a sum in ascending worker order, fp32, without the 1/N
//     factor (the caller pre-scales gradients as in Eq. 1).
//
// Pins: tests/test_oracle_*.py check this file against brute-force full sorts in
// pure Python, a hand-worked two-step example, closed forms, conservation
// invariants, numpy/torch library routines for the threshold value, the dense
// all-reduce special case (ratio = 1) and printed leader test vectors.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <iterator>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

struct Oracle {
  std::vector<int64_t> n;    // layer sizes
  std::vector<int64_t> off;  // flat offsets
  std::vector<int64_t> k;    // keep count per layer
  std::vector<int64_t> koff; // offset of the layer's segment inside a worker's list
  int64_t N = 0, K = 0;
  int32_t W = 0;
  double ratio = 1.0;
  float eps = 0.f;
  uint64_t seed = 0;
  int64_t t = 0;
  int32_t leader = -1;
  int32_t leader_override = -1;
  int threads = 0;
  float momentum = 1.0f;         // Eq. 3: the local residual enters the next step scaled by m
  bool threshold_mode = false;   // Algorithm 1 as printed: Mask <- importance > thr on the chosen node
  int32_t n_leaders = 1;         // how many chosen nodes' masks (index sets) are OR-ed
  bool per_layer_leaders = false;  // ratio mode: every layer draws its own chosen node
  std::vector<uint32_t> union_idx; // ratio mode: the index set of the last step, ascending (one node: its list)
  bool random_select = false;    // Section 3.3: elements below the threshold go with P = importance / thr
  std::vector<int32_t> leaders;  // the chosen nodes of the last step, r_1 first
  std::vector<float> thr;        // per-layer thresholds (threshold mode)
  bool layerwise = false;        // Section 3.4: thresholds from each chosen node's per-layer statistics
  double lw_alpha = 0.0, lw_beta = 0.0, lw_c = 0.0;
  std::vector<float> lw_thr;     // [chosen node][layer] thresholds of the last step (layer-wise mode)
  std::vector<uint32_t> thr_idx; // the chosen node's index set of the last step (threshold mode)
  std::vector<float> thr_val;    // its accumulated values at those indices, before zeroing
  std::vector<float> acc;        // [W][N] residuals
  std::vector<uint32_t> sel_idx; // [W][K] ascending global indices per layer segment
  std::vector<float> sel_val;    // [W][K] accumulated value at that index (before zeroing)
};

inline uint32_t bits_of(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  return u;
}

// Algorithm 1, mask line: |grad / weight|, guarded with eps.
inline float importance(float acc, float w, float eps) {
  float den = std::fabs(w) + eps;
  return std::fabs(acc) / den;
}

// keep count: ceil(n / R) in double, clamped to [1, n]
inline int64_t keep_count(int64_t n, double R) {
  double q = std::ceil(static_cast<double>(n) / R);
  int64_t k = static_cast<int64_t>(q);
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
}

inline uint64_t mix64(uint64_t z) {
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

// the randomly chosen node of step t (0-based)
inline int32_t leader_of(uint64_t seed, uint64_t t, int32_t W) {
  uint64_t z = mix64(seed + (t + 1) * 0x9E3779B97F4A7C15ull);
  uint64_t hi = z >> 32;
  return static_cast<int32_t>((hi * static_cast<uint64_t>(W)) >> 32);
}

// the chosen node of layer l at step t when every layer draws its own (Algorithm 1 draws inside the layer loop)
inline int32_t layer_leader_of(uint64_t seed, uint64_t t, uint64_t l, int32_t W) {
  uint64_t z = mix64(seed + (t + 1) * 0x9E3779B97F4A7C15ull + (l + 1) * 0xA0761D6478BD642Full);
  return static_cast<int32_t>(((z >> 32) * static_cast<uint64_t>(W)) >> 32);
}

// the chosen nodes r_1..r_n of step t: n distinct workers drawn without replacement; r_1 is leader_of()
inline std::vector<int32_t> leaders_of(uint64_t seed, uint64_t t, int32_t W, int32_t n) {
  std::vector<int32_t> remaining(W), out;
  std::iota(remaining.begin(), remaining.end(), 0);
  for (int32_t j = 0; j < n; ++j) {
    const uint64_t z = mix64(seed + (t + 1) * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(j) * 0xD1B54A32D192ED03ull);
    const uint64_t u = ((z >> 32) * static_cast<uint64_t>(W - j)) >> 32;
    out.push_back(remaining[u]);
    remaining.erase(remaining.begin() + static_cast<long>(u));
  }
  return out;
}

// Exact sum of non-negative finite doubles, rounded once (to nearest, ties to even) at the end.
// The sum is kept as a wide fixed-point number: base-2^32 digits, digit d weighing 2^(32 d - 1074),
// so that every binary64 value is an integer number of units of the lowest digit.
struct ExactSum {
  static constexpr int DIGITS = 72;
  uint64_t digit[DIGITS] = {};  // each may run ahead of 2^32 until carries are propagated
  uint32_t pending = 0;

  void carry() {
    for (int d = 0; d + 1 < DIGITS; ++d) {
      digit[d + 1] += digit[d] >> 32;
      digit[d] &= 0xffffffffull;
    }
    pending = 0;
  }
  void add(double x) {  // x >= 0, finite
    if (x == 0.0) return;
    int e;
    const double f = std::frexp(x, &e);               // x = f 2^e, 0.5 <= f < 1
    uint64_t m = static_cast<uint64_t>(std::ldexp(f, 53));  // 53-bit integer, x = m 2^(e - 53)
    int pos = e - 53 + 1074;                          // weight of m's lowest bit, in units of 2^-1074
    if (pos < 0) {                                    // subnormal: the low bits of m are zero
      m >>= -pos;
      pos = 0;
    }
    const unsigned __int128 wide = static_cast<unsigned __int128>(m) << (pos % 32);
    const int d = pos / 32;
    digit[d] += static_cast<uint64_t>(wide & 0xffffffffull);
    digit[d + 1] += static_cast<uint64_t>((wide >> 32) & 0xffffffffull);
    digit[d + 2] += static_cast<uint64_t>(wide >> 64);
    if (++pending == (1u << 30)) carry();
  }
  bool bit(int b) const { return (digit[b / 32] >> (b % 32)) & 1u; }
  double rounded() {
    carry();
    int top = -1;
    for (int b = DIGITS * 32 - 1; b >= 0; --b)
      if (bit(b)) {
        top = b;
        break;
      }
    if (top < 0) return 0.0;
    const int low = top >= 52 ? top - 52 : 0;  // lowest bit that fits the 53-bit significand
    uint64_t m = 0;
    for (int b = top; b >= low; --b) m = (m << 1) | (bit(b) ? 1u : 0u);
    if (low > 0) {
      const bool half = bit(low - 1);
      bool below = false;
      for (int b = low - 2; b >= 0 && !below; --b) below = bit(b);
      if (half && (below || (m & 1u))) m += 1;  // may reach 2^53: still exact as a double
    }
    return std::ldexp(static_cast<double>(m), low - 1074);
  }
};

// Eq. 4 for one node and layer: threshold from the exact first and second moments of the importances.
inline float layerwise_threshold(const float* acc, const float* weights, int64_t n, float eps, double alpha, double beta,
                                 double c, double* stats) {
  ExactSum s1, s2;
  for (int64_t i = 0; i < n; ++i) {
    const double imp = static_cast<double>(importance(acc[i], weights[i], eps));
    s1.add(imp);
    s2.add(imp * imp);  // exact: 24-bit significands
  }
  const double S1 = s1.rounded(), S2 = s2.rounded();
  const double nn = static_cast<double>(n);
  const double mean = S1 / nn;
  const double msq = mean * mean;
  const double var = S2 / nn - msq;
  const double v = mean > 0.0 ? var / mean : 0.0;
  const double bv = beta * v;
  const double t = v > c ? alpha + bv : alpha - bv;
  float thr = static_cast<float>(t);
  if (thr == 0.0f) thr = 0.0f;  // -0 -> +0
  if (stats) {
    stats[0] = S1;
    stats[1] = S2;
    stats[2] = mean;
    stats[3] = var;
    stats[4] = v;
  }
  return thr;
}

// Section 3.3, random gradient selection: the uniform draw of element i at step t, 24 bits
inline uint32_t draw24(uint64_t seed, uint64_t t, uint64_t i) {
  return static_cast<uint32_t>(mix64(seed + (t + 1) * 0x9E3779B97F4A7C15ull + (i + 1) * 0xC2B2AE3D27D4EB4Full) >> 40);
}

// Selection of one (worker, layer): indices (local to the layer) of the k elements
// that come first under (importance descending, index ascending), returned ascending.
void select_layer(const float* acc, const float* w, int64_t n, int64_t k, float eps,
                  std::vector<uint32_t>& keys, std::vector<uint32_t>& order) {
  keys.resize(n);
  order.resize(n);
  for (int64_t i = 0; i < n; ++i) keys[i] = bits_of(importance(acc[i], w[i], eps));
  std::iota(order.begin(), order.end(), 0u);
  auto before = [&](uint32_t a, uint32_t b) {
    if (keys[a] != keys[b]) return keys[a] > keys[b];
    return a < b;
  };
  if (k < n) std::nth_element(order.begin(), order.begin() + (k - 1), order.end(), before);
  order.resize(k);
  std::sort(order.begin(), order.end());
}

}  // namespace

extern "C" {

int32_t oracle_leader(uint64_t seed, uint64_t t, int32_t W) { return leader_of(seed, t, W); }
uint64_t oracle_mix64(uint64_t z) { return mix64(z); }
int64_t oracle_keep_count(int64_t n, double R) { return keep_count(n, R); }
uint32_t oracle_importance_bits(float acc, float w, float eps) { return bits_of(importance(acc, w, eps)); }

// Stand-alone selection of one layer (used by the brute-force pins).
void oracle_select(const float* acc, const float* w, int64_t n, int64_t k, float eps, uint32_t* out_idx) {
  std::vector<uint32_t> keys, order;
  select_layer(acc, w, n, k, eps, keys, order);
  std::copy(order.begin(), order.end(), out_idx);
}

void* oracle_create(const int64_t* layer_sizes, int32_t n_layers, int32_t W, double ratio, float eps,
                    uint64_t seed) {
  if (!layer_sizes || n_layers < 1 || W < 1 || !(ratio >= 1.0) || !std::isfinite(ratio) || !(eps > 0.f) ||
      !std::isfinite(eps))
    return nullptr;
  Oracle* o = new Oracle;
  o->W = W;
  o->ratio = ratio;
  o->eps = eps;
  o->seed = seed;
  for (int32_t l = 0; l < n_layers; ++l) {
    if (layer_sizes[l] < 1) {
      delete o;
      return nullptr;
    }
    o->n.push_back(layer_sizes[l]);
    o->off.push_back(o->N);
    o->k.push_back(keep_count(layer_sizes[l], ratio));
    o->koff.push_back(o->K);
    o->N += layer_sizes[l];
    o->K += o->k.back();
  }
  if (o->N >= (int64_t(1) << 32)) {
    delete o;
    return nullptr;
  }
  o->acc.assign(static_cast<size_t>(W) * o->N, 0.0f);
  o->sel_idx.assign(static_cast<size_t>(W) * o->K, 0u);
  o->sel_val.assign(static_cast<size_t>(W) * o->K, 0.0f);
  return o;
}

void oracle_destroy(void* h) { delete static_cast<Oracle*>(h); }

void oracle_set_threads(void* h, int32_t threads) { static_cast<Oracle*>(h)->threads = threads; }
int32_t oracle_threads_used(void* h) {
#ifdef _OPENMP
  Oracle* o = static_cast<Oracle*>(h);
  return o->threads > 0 ? o->threads : omp_get_max_threads();
#else
  (void)h;
  return 1;
#endif
}
// Switches to Algorithm 1 as printed, with one absolute threshold per layer (NULL: back to the ratio).
void oracle_set_thresholds(void* h, const float* thr) {
  Oracle* o = static_cast<Oracle*>(h);
  o->threshold_mode = thr != nullptr;
  if (thr) o->thr.assign(thr, thr + o->n.size());
}
// Section 3.4: thresholds from the chosen nodes' own statistics (switches the threshold mode on as well).
void oracle_set_layerwise(void* h, int32_t on, double alpha, double beta, double c) {
  Oracle* o = static_cast<Oracle*>(h);
  o->layerwise = on != 0;
  o->lw_alpha = alpha;
  o->lw_beta = beta;
  o->lw_c = c;
  if (on) {
    o->threshold_mode = true;
    o->thr.assign(o->n.size(), 0.0f);
  }
}
// [chosen node][layer] thresholds the last step derived; returns how many chosen nodes there were
int32_t oracle_get_layer_thresholds(void* h, float* out) {
  Oracle* o = static_cast<Oracle*>(h);
  std::copy(o->lw_thr.begin(), o->lw_thr.end(), out);
  return static_cast<int32_t>(o->lw_thr.size() / o->n.size());
}
// the pieces of Eq. 4 on their own (tests): exact sum of non-negative doubles; one layer's statistics
double oracle_exact_sum(const double* x, int64_t n) {
  ExactSum s;
  for (int64_t i = 0; i < n; ++i) s.add(x[i]);
  return s.rounded();
}
float oracle_layerwise_threshold(const float* acc, const float* weights, int64_t n, float eps, double alpha, double beta,
                                 double c, double* stats5) {
  return layerwise_threshold(acc, weights, n, eps, alpha, beta, c, stats5);
}
void oracle_set_random_select(void* h, int32_t on) { static_cast<Oracle*>(h)->random_select = on != 0; }
uint32_t oracle_draw24(uint64_t seed, uint64_t t, uint64_t i) { return draw24(seed, t, i); }
void oracle_set_n_leaders(void* h, int32_t n) { static_cast<Oracle*>(h)->n_leaders = n; }
void oracle_leaders(uint64_t seed, uint64_t t, int32_t W, int32_t n, int32_t* out) {
  const std::vector<int32_t> v = leaders_of(seed, t, W, n);
  std::copy(v.begin(), v.end(), out);
}
int64_t oracle_threshold_list_length(void* h) { return static_cast<int64_t>(static_cast<Oracle*>(h)->thr_idx.size()); }
void oracle_get_threshold_list(void* h, uint32_t* idx, float* val) {
  Oracle* o = static_cast<Oracle*>(h);
  std::copy(o->thr_idx.begin(), o->thr_idx.end(), idx);
  std::copy(o->thr_val.begin(), o->thr_val.end(), val);
}
void oracle_set_momentum(void* h, float m) { static_cast<Oracle*>(h)->momentum = m; }
void oracle_set_per_layer_leaders(void* h, int32_t on) { static_cast<Oracle*>(h)->per_layer_leaders = on != 0; }
int32_t oracle_layer_leader(uint64_t seed, uint64_t t, uint64_t l, int32_t W) { return layer_leader_of(seed, t, l, W); }
void oracle_set_leader_override(void* h, int32_t leader) { static_cast<Oracle*>(h)->leader_override = leader; }
int64_t oracle_total(void* h) { return static_cast<Oracle*>(h)->N; }
int64_t oracle_total_keep(void* h) { return static_cast<Oracle*>(h)->K; }
int64_t oracle_get_step(void* h) { return static_cast<Oracle*>(h)->t; }
int32_t oracle_get_leader(void* h) { return static_cast<Oracle*>(h)->leader; }

void oracle_get_layout(void* h, int64_t* off, int64_t* k) {
  Oracle* o = static_cast<Oracle*>(h);
  for (size_t l = 0; l < o->n.size(); ++l) {
    off[l] = o->off[l];
    k[l] = o->k[l];
  }
}

void oracle_reset(void* h) {
  Oracle* o = static_cast<Oracle*>(h);
  std::fill(o->acc.begin(), o->acc.end(), 0.0f);
  o->t = 0;
  o->leader = -1;
}

void oracle_set_residual(void* h, int32_t w, const float* src) {
  Oracle* o = static_cast<Oracle*>(h);
  std::memcpy(&o->acc[static_cast<size_t>(w) * o->N], src, sizeof(float) * o->N);
}

void oracle_get_residual(void* h, int32_t w, float* dst) {
  Oracle* o = static_cast<Oracle*>(h);
  std::memcpy(dst, &o->acc[static_cast<size_t>(w) * o->N], sizeof(float) * o->N);
}

void oracle_get_selection(void* h, int32_t w, uint32_t* idx, float* val) {
  Oracle* o = static_cast<Oracle*>(h);
  std::memcpy(idx, &o->sel_idx[static_cast<size_t>(w) * o->K], sizeof(uint32_t) * o->K);
  std::memcpy(val, &o->sel_val[static_cast<size_t>(w) * o->K], sizeof(float) * o->K);
}

// one byte per element, 1 where the element is in the index set of the last step
void oracle_get_mask(void* h, uint8_t* dst) {
  Oracle* o = static_cast<Oracle*>(h);
  std::memset(dst, 0, o->N);
  if (o->leader < 0) return;
  if (o->threshold_mode) {
    for (uint32_t i : o->thr_idx) dst[i] = 1;
    return;
  }
  for (uint32_t i : o->union_idx) dst[i] = 1;
}

// ratio mode: the index set of the last step (the union of the chosen nodes' lists), ascending
int64_t oracle_union_length(void* h) { return static_cast<int64_t>(static_cast<Oracle*>(h)->union_idx.size()); }
void oracle_get_union(void* h, uint32_t* idx) {
  Oracle* o = static_cast<Oracle*>(h);
  std::copy(o->union_idx.begin(), o->union_idx.end(), idx);
}

// One step.  grads[W][N], weights[N], update[N]: host pointers.
void oracle_step(void* h, const float* grads, const float* weights, float* update) {
  Oracle* o = static_cast<Oracle*>(h);
  const int64_t N = o->N, K = o->K;
  const int32_t W = o->W;
  const int L = static_cast<int>(o->n.size());
#ifdef _OPENMP
  const int nthreads = o->threads > 0 ? o->threads : omp_get_max_threads();
#endif

  // (a) accumulate the new gradient into the local residual; with momentum (Eq. 3,
  // s_t = sparse(m g_{t-1} + g_t)) what was kept locally is first scaled by m: one rounded
  // product, then one rounded sum (m = 1 leaves the residual unchanged)
  const float m = o->momentum;
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t e = 0; e < static_cast<int64_t>(W) * N; ++e) {
    const float carried = m * o->acc[e];
    o->acc[e] = carried + grads[e];
  }

  o->leader = o->leader_override >= 0 ? o->leader_override : leader_of(o->seed, static_cast<uint64_t>(o->t), W);
  if (o->threshold_mode) {
    // Algorithm 1 as printed: the chosen node r alone forms Mask_r = |G_r / w| > thr, layer by layer;
    // every node then splits its accumulated gradient by that mask
    // with n > 1 chosen nodes the masks are OR-ed (Algorithm 1: Mask = OR Mask_{r_i})
    if (o->leader_override >= 0 || o->n_leaders == 1) {
      o->leaders.assign(1, o->leader);
    } else {
      o->leaders = leaders_of(o->seed, static_cast<uint64_t>(o->t), W, o->n_leaders);
    }
    const float* ar = &o->acc[static_cast<size_t>(o->leader) * N];
    o->thr_idx.clear();
    o->thr_val.clear();
    const int n_chosen = static_cast<int>(o->leaders.size());
    if (o->layerwise) {  // Section 3.4: every chosen node derives its own per-layer thresholds
      o->lw_thr.assign(static_cast<size_t>(n_chosen) * L, 0.0f);
#pragma omp parallel for num_threads(nthreads) schedule(dynamic, 1)
      for (int q = 0; q < n_chosen * L; ++q) {
        const int j = q / L, l = q % L;
        o->lw_thr[q] = layerwise_threshold(&o->acc[static_cast<size_t>(o->leaders[j]) * N + o->off[l]], weights + o->off[l],
                                           o->n[l], o->eps, o->lw_alpha, o->lw_beta, o->lw_c, nullptr);
      }
    }
    for (int l = 0; l < L; ++l) {
      for (int64_t i = o->off[l]; i < o->off[l] + o->n[l]; ++i) {
        bool in_mask = false;
        for (int j = 0; j < n_chosen; ++j) {
          const int32_t r = o->leaders[j];
          const float thr_l = o->layerwise ? o->lw_thr[static_cast<size_t>(j) * L + l] : o->thr[l];
          const float imp = importance(o->acc[static_cast<size_t>(r) * N + i], weights[i], o->eps);
          bool sel = imp > thr_l;
          if (!sel && o->random_select) {
            // P(update) = importance / threshold: one draw per element and step, compared in fp32
            const float u = static_cast<float>(draw24(o->seed, static_cast<uint64_t>(o->t), static_cast<uint64_t>(i))) *
                            5.9604644775390625e-08f;  // 2^-24
            sel = u < imp / thr_l;
          }
          in_mask = in_mask || sel;
        }
        if (in_mask) {
          o->thr_idx.push_back(static_cast<uint32_t>(i));
          o->thr_val.push_back(ar[i]);  // listed values are r_1's
        }
      }
    }
    for (int64_t i = 0; i < N; ++i) update[i] = 0.0f;
    for (size_t j = 0; j < o->thr_idx.size(); ++j) {
      const size_t i = o->thr_idx[j];
      float s = o->acc[i];
      for (int32_t w = 1; w < W; ++w) s = s + o->acc[static_cast<size_t>(w) * N + i];
      update[i] = 0.0f + s;
    }
    for (size_t j = 0; j < o->thr_idx.size(); ++j)
      for (int32_t w = 0; w < W; ++w) o->acc[static_cast<size_t>(w) * N + o->thr_idx[j]] = 0.0f;
    o->t += 1;
    return;
  }

  // (b)-(d) per worker and layer: importance, keep the k best, list them in index order
#pragma omp parallel num_threads(nthreads)
  {
    std::vector<uint32_t> keys, order;
#pragma omp for schedule(dynamic, 1)
    for (int64_t p = 0; p < static_cast<int64_t>(W) * L; ++p) {
      // large layers first within a worker does not matter for correctness
      const int32_t w = static_cast<int32_t>(p / L);
      const int l = static_cast<int>(p % L);
      const float* a = &o->acc[static_cast<size_t>(w) * N + o->off[l]];
      select_layer(a, weights + o->off[l], o->n[l], o->k[l], o->eps, keys, order);
      uint32_t* li = &o->sel_idx[static_cast<size_t>(w) * K + o->koff[l]];
      float* lv = &o->sel_val[static_cast<size_t>(w) * K + o->koff[l]];
      for (int64_t j = 0; j < o->k[l]; ++j) {
        li[j] = static_cast<uint32_t>(o->off[l] + order[j]);
        lv[j] = a[order[j]];
      }
    }
  }

  // (e) the randomly chosen node supplies the index set; with several chosen nodes (Algorithm 1:
  // Mask = OR Mask_{r_i}) it is the union of their lists, ascending, each index once
  if (o->leader_override >= 0 || o->n_leaders == 1) {
    o->leaders.assign(1, o->leader);
  } else {
    o->leaders = leaders_of(o->seed, static_cast<uint64_t>(o->t), W, o->n_leaders);
  }
  o->union_idx.clear();
  if (o->per_layer_leaders && o->leader_override < 0 && o->n_leaders == 1) {
    // every layer takes its own chosen node's segment of that node's list
    for (int l = 0; l < L; ++l) {
      const int32_t r = layer_leader_of(o->seed, static_cast<uint64_t>(o->t), static_cast<uint64_t>(l), W);
      const uint32_t* list = &o->sel_idx[static_cast<size_t>(r) * K + o->koff[l]];
      o->union_idx.insert(o->union_idx.end(), list, list + o->k[l]);
    }
    o->leaders.clear();
  }
  for (int32_t r : o->leaders) {
    const uint32_t* list = &o->sel_idx[static_cast<size_t>(r) * K];
    std::vector<uint32_t> merged;
    std::set_union(o->union_idx.begin(), o->union_idx.end(), list, list + K, std::back_inserter(merged));
    o->union_idx.swap(merged);
  }
  const uint32_t* S = o->union_idx.data();
  const int64_t n_set = static_cast<int64_t>(o->union_idx.size());

  // (f) sum over workers in ascending order at the shared indices, into a zeroed dense update
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t i = 0; i < N; ++i) update[i] = 0.0f;
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t j = 0; j < n_set; ++j) {
    const size_t i = S[j];
    float s = o->acc[i];
    for (int32_t w = 1; w < W; ++w) s = s + o->acc[static_cast<size_t>(w) * N + i];
    update[i] = 0.0f + s;
  }

  // (g) what was sent leaves every worker's residual; the rest stays
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t j = 0; j < n_set; ++j) {
    const size_t i = S[j];
    for (int32_t w = 0; w < W; ++w) o->acc[static_cast<size_t>(w) * N + i] = 0.0f;
  }
  o->t += 1;
}

}  // extern "C"

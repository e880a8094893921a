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
//   * one randomly chosen node per step supplies the index set (Section 3.2:
//     "randomly choose a node and broadcast its important gradient index").
//   * Eq. 3's momentum acts on the locally kept residual: G <- m * G + grad (two roundings);
//     m = 1, the default, is the plain accumulation of Section 3.2.
//   * threshold mode is Algorithm 1 as printed: only the chosen node forms a mask, per layer
//     Mask = importance > thr[layer] (strict), the index set has whatever size results, and no
//     other worker makes a selection of its own.
//   * Section 3.3's random gradient selection (threshold mode, optional): an element whose importance
//     does not exceed the threshold is sent iff u < importance / thr, u one 24-bit uniform draw per
//     element and step, the quotient in fp32.
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
  int32_t n_leaders = 1;         // threshold mode: how many chosen nodes' masks are OR-ed
  bool random_select = false;    // Section 3.3: elements below the threshold go with P = importance / thr
  std::vector<int32_t> leaders;  // the chosen nodes of the last step, r_1 first
  std::vector<float> thr;        // per-layer thresholds (threshold mode)
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
  const uint32_t* S = &o->sel_idx[static_cast<size_t>(o->leader) * o->K];
  for (int64_t j = 0; j < o->K; ++j) dst[S[j]] = 1;
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
    for (int l = 0; l < L; ++l) {
      for (int64_t i = o->off[l]; i < o->off[l] + o->n[l]; ++i) {
        bool in_mask = false;
        for (int32_t r : o->leaders) {
          const float imp = importance(o->acc[static_cast<size_t>(r) * N + i], weights[i], o->eps);
          bool sel = imp > o->thr[l];
          if (!sel && o->random_select) {
            // P(update) = importance / threshold: one draw per element and step, compared in fp32
            const float u = static_cast<float>(draw24(o->seed, static_cast<uint64_t>(o->t), static_cast<uint64_t>(i))) *
                            5.9604644775390625e-08f;  // 2^-24
            sel = u < imp / o->thr[l];
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

  // (e) the randomly chosen node supplies the index set
  const uint32_t* S = &o->sel_idx[static_cast<size_t>(o->leader) * K];

  // (f) sum over workers in ascending order at the shared indices, into a zeroed dense update
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t i = 0; i < N; ++i) update[i] = 0.0f;
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t j = 0; j < K; ++j) {
    const size_t i = S[j];
    float s = o->acc[i];
    for (int32_t w = 1; w < W; ++w) s = s + o->acc[static_cast<size_t>(w) * N + i];
    update[i] = 0.0f + s;
  }

  // (g) what was sent leaves every worker's residual; the rest stays
#pragma omp parallel for num_threads(nthreads) schedule(static)
  for (int64_t j = 0; j < K; ++j) {
    const size_t i = S[j];
    for (int32_t w = 0; w < W; ++w) o->acc[static_cast<size_t>(w) * N + i] = 0.0f;
  }
  o->t += 1;
}

}  // extern "C"

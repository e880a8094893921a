// Absolute-threshold mode (Algorithm 1 as printed), random sub-threshold selection (Section 3.3) and the
// layer-wise threshold from exact moments (Section 3.4, Eq. 4).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_device.cuh"
#include "iwp_stream.cuh"

namespace iwp {

// ---------------------------------------------------------------------------------------
// Absolute-threshold mode: Algorithm 1 as printed.  Only the chosen nodes form masks, per layer
// Mask = |G / w| > thr (strict; several nodes' masks are OR-ed), and the index set has whatever size
// results.  A step: step (a) for the chosen nodes (inside k_thr_mask_count, or k_thr_stats with layer-wise
// thresholds), two looks at their
// residuals - count per chunk, scan, stable compaction with one set bit per element - and one
// streaming pass over all workers that does the rest (k_thr_fused).  thr_bits: the thresholds' fp32
// patterns; a negative one (the layer-wise rule can produce it) passes everything, +inf nothing.
// ---------------------------------------------------------------------------------------
// Random selection parameters of a step (Section 3.3): off, or the seed and step of the draws.
struct RandomSelect {
  int on;
  uint64_t seed;
  uint64_t step;
};

// Mask bit of one element on one chosen node: importance > thr, or - with random selection on - a
// draw below importance / thr (P(update) = importance / threshold; one draw per element and step).
// gm, gme: the multiply pre-test of the streaming pass (pretest_multiplier(T, eps) and its product with eps):
// an element whose exactly rounded quotient exceeds T passes |acc| >= gm (|w| + eps), so without random
// selection everything that fails it is out without a division.
__device__ __forceinline__ bool thr_selected(float acc, float w, float eps, uint32_t T, float gm, float gme, uint64_t e,
                                             const RandomSelect& rs) {
  if (!rs.on && !(fabsf(acc) >= __fmaf_rn(gm, fabsf(w), gme))) return false;
  const uint32_t key = imp_key(acc, w, eps);
  // importance patterns are non-negative, so as signed integers they order like the values against any
  // threshold pattern: a negative threshold (layer-wise mode can produce one) is below every importance
  if (static_cast<int32_t>(key) > static_cast<int32_t>(T)) return true;
  if (!rs.on) return false;
  const float u = __fmul_rn(static_cast<float>(draw24(rs.seed, rs.step, e)), 5.9604644775390625e-08f);
  return u < __fdiv_rn(__uint_as_float(key), __uint_as_float(T));
}

// First look at the chosen nodes' residuals, chunk by chunk: (ACCUMULATE: step (a) for them, acc <- m acc + g,
// on the way;) the OR of their masks as one bit per element (`set_bits`, zeroed before the step) and the
// number of set elements of the chunk.  Everything after this pass works from the bits.  grid = chunks.
template <bool VEC, bool ACCUMULATE>
__global__ void __launch_bounds__(THREADS)
    k_thr_mask_count(const float* __restrict__ grads, float* __restrict__ acc, const float* __restrict__ weights,
                     const Chunk* __restrict__ chunks, const uint32_t* __restrict__ thr_bits, uint32_t thr_stride,
                     uint32_t* __restrict__ set_bits, uint32_t* __restrict__ chunk_cnt, float eps, uint64_t N,
                     float momentum, LeaderSet ls, RandomSelect rs) {
  __shared__ uint32_t sh_cnt;
  const Chunk c = chunks[blockIdx.x];
  // thr_stride = 0: one threshold per layer for every chosen node; = number of layers: node j has its own row
  const uint32_t* T = thr_bits + c.layer;
  __shared__ float sh_gm[MAX_LEADERS];  // pre-test multiplier of every chosen node's threshold
  if (threadIdx.x == 0) sh_cnt = 0;
  if (threadIdx.x < ls.n) sh_gm[threadIdx.x] = pretest_multiplier(T[threadIdx.x * thr_stride], eps);
  __syncthreads();
  const uint64_t lo = c.a, hi = lo + c.len;
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  uint32_t cnt = 0;
  constexpr int U = 2;  // slots per thread and trip: the loads of both are issued before either is used
  for (uint32_t it = 0; it < n_iter; it += U) {
    uint64_t e0[U];
    float wv[U][4];
    uint32_t f[U];  // Mask = OR of the chosen nodes' masks
#pragma unroll
    for (int u = 0; u < U; ++u) {
      e0[u] = s0 + (static_cast<uint64_t>(it + u) * THREADS + threadIdx.x) * 4;  // beyond the chunk: every access is guarded
      load4<VEC>(weights, e0[u], lo, hi, wv[u]);
      f[u] = 0;
    }
    for (int j = 0; j < ls.n; ++j) {
      float* a = acc + static_cast<uint64_t>(ls.r[j]) * N;
      const float* g = grads + static_cast<uint64_t>(ls.r[j]) * N;
      const float gm = sh_gm[j], gme = __fmul_rn(gm, eps);
      const uint32_t Tj = T[j * thr_stride];
      float av[U][4], gv[U][4];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        load4_stream<VEC>(a, e0[u], lo, hi, av[u]);
        if (ACCUMULATE) load4_stream<VEC>(g, e0[u], lo, hi, gv[u]);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (ACCUMULATE) {
#pragma unroll
          for (int q = 0; q < 4; ++q) av[u][q] = accumulate(av[u][q], gv[u][q], momentum);
          store4<VEC>(a, e0[u], lo, hi, av[u]);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
          f[u] |= thr_selected(av[u][q], wv[u][q], eps, Tj, gm, gme, e0[u] + q, rs) ? (1u << q) : 0u;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      uint32_t inside = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) inside |= (e0[u] + q >= lo && e0[u] + q < hi) ? (1u << q) : 0u;
      f[u] &= inside;
      // a slot's four bits never straddle a word because slots start at multiples of four
      if (f[u]) atomicOr(&set_bits[e0[u] >> 5], f[u] << (e0[u] & 31u));
      cnt += __popc(f[u]);
    }
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
  if ((threadIdx.x & 31) == 0 && cnt) atomicAdd(&sh_cnt, cnt);
  __syncthreads();
  if (threadIdx.x == 0) chunk_cnt[blockIdx.x] = sh_cnt;
}

// Exclusive prefix sum of the chunk counts (chunks are in index order) and the list length.
// One CTA of 1024 threads walks the chunks 1024 at a time.
__global__ void __launch_bounds__(1024)
    k_thr_scan(const uint32_t* __restrict__ chunk_cnt, uint32_t* __restrict__ chunk_off, uint32_t n_chunks,
               uint32_t* __restrict__ list_len) {
  __shared__ uint32_t sh_w[32];
  __shared__ uint32_t sh_run;
  if (threadIdx.x == 0) sh_run = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (uint32_t base = 0; base < n_chunks; base += 1024) {
    const uint32_t j = base + threadIdx.x;
    const uint32_t v = j < n_chunks ? chunk_cnt[j] : 0u;
    const uint32_t incl = warp_incl_scan(v);
    if (lane == 31) sh_w[wid] = incl;
    __syncthreads();
    uint32_t woff = 0, tot = 0;
    for (int i = 0; i < 32; ++i) {
      const uint32_t x = sh_w[i];
      if (i < wid) woff += x;
      tot += x;
    }
    const uint32_t run = sh_run;
    if (j < n_chunks) chunk_off[j] = run + woff + incl - v;
    __syncthreads();
    if (threadIdx.x == 0) sh_run = run + tot;
    __syncthreads();
  }
  if (threadIdx.x == 0) *list_len = sh_run;
}

// Second look, from the bits alone: the ordered index list (ascending; offsets from the scan of the chunk
// counts) with r_1's residuals as the listed values, read only where a bit is set.  grid = chunks.
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_thr_write(const float* __restrict__ acc_r1, const Chunk* __restrict__ chunks, const uint32_t* __restrict__ chunk_off,
                const uint32_t* __restrict__ set_bits, uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val,
                uint32_t capacity, int* __restrict__ status) {
  __shared__ uint32_t sh_warp[WARPS];
  const Chunk c = chunks[blockIdx.x];
  uint32_t run = chunk_off[blockIdx.x];
  const uint64_t lo = c.a, hi = lo + c.len;
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  for (uint32_t it = 0; it < n_iter; ++it) {
    const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
    // the bits of neighbouring layers in the same word belong to other chunks: keep this chunk's elements only
    uint32_t f = (e0 < hi) ? (set_bits[e0 >> 5] >> (e0 & 31u)) & 0xFu : 0u;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (e0 + q < lo || e0 + q >= hi) f &= ~(1u << q);
    float av[4] = {0.f, 0.f, 0.f, 0.f};
    if (f) load4<VEC>(acc_r1, e0, lo, hi, av);
    uint32_t total;
    uint32_t pos = run + block_excl_scan(static_cast<uint32_t>(__popc(f)), sh_warp, total);
    if (f) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if ((f >> q) & 1u) {
          if (pos < capacity) {
            sel_idx[pos] = static_cast<uint32_t>(e0 + q);
            sel_val[pos] = av[q];
          } else {
            atomicMin(status, STATUS_CAPACITY);
          }
          ++pos;
        }
      }
    }
    run += total;
  }
}

// ---------------------------------------------------------------------------------------
// Layer-wise threshold (Section 3.4, Eq. 4): thr = alpha + beta v if v > C else alpha - beta v with
// v = var / mean of the layer's importances on a chosen node.  The two moments are defined as EXACT
// sums rounded once to binary64, so that no summation order enters the result.  An importance is
// m 2^(f - 150) with a 24-bit integer m and f = max(biased exponent, 1); per biased exponent the
// kernel below sums m, and the two 24-bit halves of m^2, in 64-bit integers (no rounding anywhere);
// k_thr_finalize then adds the bins up as wide integers, rounds once and evaluates Eq. 4 in binary64.
// Moment bins: [chosen node][layer][3][256] (sum m | sum m^2 >> 24 | sum m^2 & 0xffffff).
// ---------------------------------------------------------------------------------------
constexpr int LW_BINS = 384;  // 255 exponents, plus room for the 32-bit digits of the per-CTA sums (see below)

// One (chunk, chosen node) per CTA; grid = (chunks, chosen nodes).
// Fast path: the CTA picks a window of 31 binades around the average exponent of its first elements;
// an importance m 2^(f - 150) with f - base = d in the window is added as the integer m << d (and
// m^2 << 2d) to per-thread 64-bit (128-bit) sums, which cannot overflow for the at most 2^9 elements a
// thread sees; the threads' sums are added up digit by digit (base 2^32) and each digit goes to the
// bin whose weight it has: digit k of the first moment to bin base + 32 k, of the second to bin
// base + 16 k (a bin index step doubles the weight of m and quadruples that of m^2).
// Slow path, for the few elements outside the window: lanes with the same exponent add their terms
// with one warp reduction and one shared-memory atomic per term.
constexpr uint32_t STATS_GROUP = 1;  // chunks per CTA of k_thr_stats (more were measured slower: the pass wants many CTAs)

// ACCUM: the pass is also step (a) for the chosen nodes (it reads their gradients and writes their residuals back),
// which saves the separate accumulate pass over them.
template <bool VEC, bool ACCUM>
__global__ void __launch_bounds__(THREADS)
    k_thr_stats(float* __restrict__ acc, const float* __restrict__ grads, const float* __restrict__ weights,
                const Chunk* __restrict__ chunks, uint32_t n_chunks, unsigned long long* __restrict__ bins, float eps,
                uint64_t N, uint32_t n_layers, float momentum, LeaderSet ls) {
  __shared__ unsigned long long sh[3 * LW_BINS];
  __shared__ uint32_t sh_exp[2];  // sum and count of the exponents sampled for the window
  const int j = blockIdx.y;
  int r = ls.r[0];
#pragma unroll
  for (int q = 1; q < MAX_LEADERS; ++q)
    if (q == j) r = ls.r[q];
  float* a = acc + static_cast<uint64_t>(r) * N;
  const float* g = grads + static_cast<uint64_t>(r) * N;
  const int lane = threadIdx.x & 31;
  for (int b = threadIdx.x; b < 3 * LW_BINS; b += THREADS) sh[b] = 0ull;
  auto flush = [&](uint32_t layer) {  // this CTA's bins of one layer into the global ones; leaves them cleared
    __syncthreads();
    unsigned long long* g = bins + (static_cast<uint64_t>(j) * n_layers + layer) * (3 * LW_BINS);
    for (int b = threadIdx.x; b < 3 * LW_BINS; b += THREADS) {
      const unsigned long long v = sh[b];
      if (v) {
        atomicAdd(&g[b], v);
        sh[b] = 0ull;
      }
    }
    __syncthreads();
  };
  // a group of consecutive chunks per CTA: the bins are shared by the chunks of a layer and go to global
  // memory when the layer changes and at the end
  const uint32_t c_first = blockIdx.x * STATS_GROUP, c_last = min(c_first + STATS_GROUP, n_chunks);
  uint32_t cur_layer = chunks[c_first].layer;
  for (uint32_t ci = c_first; ci < c_last; ++ci) {
    const Chunk c = chunks[ci];
    if (c.layer != cur_layer) {
      flush(cur_layer);
      cur_layer = c.layer;
    }
    if (threadIdx.x < 2) sh_exp[threadIdx.x] = 0u;
    __syncthreads();
    const uint64_t lo = c.a, hi = lo + c.len;
    const uint64_t s0 = lo & ~3ull;
    const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
    // widest shift that keeps m << d inside 63 bits summed over this thread's elements (and m^2 << 2d inside 127)
    const int d_max = min(30, 39 - (32 - __clz(n_iter * 4)));
    int base = 1;
    {  // window: average exponent of the first element of every thread, minus 14
      const uint64_t e = s0 + static_cast<uint64_t>(threadIdx.x) * 4;
      uint32_t f = 0, cnt = 0;
      for (int q = 0; q < 4 && cnt == 0; ++q) {
        if (e + q >= lo && e + q < hi) {
          const float v = ACCUM ? accumulate(a[e + q], g[e + q], momentum) : a[e + q];  // (not stored yet: read only)
          const uint32_t key = imp_key(v, weights[e + q], eps);
          if (key != 0u && key < 0x7f800000u) {
            f = max(key >> 23, 1u);
            cnt = 1;
          }
        }
      }
      f = __reduce_add_sync(0xffffffffu, f);
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (lane == 0 && cnt) {
        atomicAdd(&sh_exp[0], f);
        atomicAdd(&sh_exp[1], cnt);
      }
      __syncthreads();
      if (sh_exp[1]) base = max(1, static_cast<int>(sh_exp[0] / sh_exp[1]) - 14);
    }
    unsigned long long s1 = 0ull;
    unsigned __int128 s2 = 0;
    for (uint32_t it = 0; it < n_iter; ++it) {
      const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
      float av[4], wv[4];
      load4<VEC>(a, e0, lo, hi, av);
      load4<VEC>(weights, e0, lo, hi, wv);
      if (ACCUM) {
        float gv[4];
        load4_stream<VEC>(g, e0, lo, hi, gv);
#pragma unroll
        for (int q = 0; q < 4; ++q) av[q] = accumulate(av[q], gv[q], momentum);
        store4<VEC>(a, e0, lo, hi, av);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t e = e0 + q;
        const uint32_t key = imp_key(av[q], wv[q], eps);
        // zero adds nothing; a non-finite importance is outside the contract and is left out
        bool valid = e >= lo && e < hi && key != 0u && key < 0x7f800000u;
        const uint32_t ex = key >> 23;
        const uint32_t m = ex ? ((key & 0x7fffffu) | 0x800000u) : key;
        const unsigned long long m2 = static_cast<unsigned long long>(m) * m;
        const int d = static_cast<int>(max(ex, 1u)) - base;
        if (valid && d >= 0 && d <= d_max) {
          s1 += static_cast<unsigned long long>(m) << d;
          s2 += static_cast<unsigned __int128>(m2) << (2 * d);
          valid = false;
        }
        unsigned todo = __ballot_sync(0xffffffffu, valid);
        if (todo == 0u) continue;
        const uint32_t h = static_cast<uint32_t>(m2 >> 24), l = static_cast<uint32_t>(m2) & 0xffffffu;
        while (todo) {
          const int first = __ffs(todo) - 1;
          const uint32_t ex_first = __shfl_sync(0xffffffffu, ex, first);
          const bool mine = valid && ex == ex_first;
          const unsigned grp = __ballot_sync(0xffffffffu, mine);
          if (mine) {  // 32 terms below 2^24 fit 32 bits
            const uint32_t sm = __reduce_add_sync(grp, m), shh = __reduce_add_sync(grp, h), sl = __reduce_add_sync(grp, l);
            if (lane == first) {
              atomicAdd(&sh[ex_first], static_cast<unsigned long long>(sm));
              atomicAdd(&sh[LW_BINS + ex_first], static_cast<unsigned long long>(shh));
              atomicAdd(&sh[2 * LW_BINS + ex_first], static_cast<unsigned long long>(sl));
            }
          }
          todo &= ~grp;
        }
      }
    }
    // the thread's window sums, digit by digit, into the bins whose weight the digits have: digit k of the
    // first moment is worth bin base + 32 k, of the second bin base + 16 k (see above)
    if (s1) {
      atomicAdd(&sh[base], s1 & 0xffffffffull);
      atomicAdd(&sh[base + 32], s1 >> 32);
    }
    if (s2) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const unsigned long long dg = static_cast<unsigned long long>(s2 >> (32 * k)) & 0xffffffffull;
        if (dg) atomicAdd(&sh[2 * LW_BINS + base + 16 * k], dg);
      }
    }
  }
  flush(cur_layer);
}

// The wide integer in base-2^32 digits (64-bit words that may run ahead until the carries are
// propagated here) times 2^unit_exp, rounded to nearest even binary64.
__device__ inline double lw_round(unsigned long long* digit, int n_digits, int unit_exp) {
  for (int d = 0; d + 1 < n_digits; ++d) {
    digit[d + 1] += digit[d] >> 32;
    digit[d] &= 0xffffffffull;
  }
  int td = n_digits - 1;
  while (td >= 0 && digit[td] == 0ull) --td;
  if (td < 0) return 0.0;
  // the three leading digits hold the 53 bits to keep, the bit that decides and some of the rest
  const unsigned __int128 X = (static_cast<unsigned __int128>(digit[td]) << 64) |
                              (static_cast<unsigned __int128>(td >= 1 ? digit[td - 1] : 0ull) << 32) |
                              static_cast<unsigned __int128>(td >= 2 ? digit[td - 2] : 0ull);
  const int drop = 64 + 31 - __clz(static_cast<unsigned>(digit[td])) - 52;  // >= 12 bits go
  unsigned long long m = static_cast<unsigned long long>(X >> drop);
  if ((X >> (drop - 1)) & 1) {
    bool below = (X & ((static_cast<unsigned __int128>(1) << (drop - 1)) - 1)) != 0;
    for (int d = td - 3; d >= 0 && !below; --d) below = digit[d] != 0ull;
    if (below || (m & 1ull)) m += 1;  // may reach 2^53: still exact
  }
  return ldexp(static_cast<double>(m), 32 * (td - 2) + drop + unit_exp);
}

// Eq. 4 per (layer, chosen node): grid = (layers, chosen nodes).  Every thread adds its bins, shifted
// to their weight, into the two wide sums in shared memory; one thread rounds and does the binary64
// arithmetic; the bins are cleared for the next step.
__global__ void __launch_bounds__(THREADS)
    k_thr_finalize(unsigned long long* __restrict__ bins, const LayerDesc* __restrict__ layers, uint32_t* __restrict__ thr_bits,
                   uint32_t n_layers, double alpha, double beta, double c_split) {
  constexpr int D1 = 16, D2 = 32;  // digits: 64 + 383 bits for the first moment, 64 + 24 + 766 for the second
  __shared__ unsigned long long d1[D1], d2[D2];
  const uint32_t layer = blockIdx.x, j = blockIdx.y;
  unsigned long long* g = bins + (static_cast<uint64_t>(j) * n_layers + layer) * (3 * LW_BINS);
  if (threadIdx.x < D1) d1[threadIdx.x] = 0ull;
  if (threadIdx.x < D2) d2[threadIdx.x] = 0ull;
  __syncthreads();
  for (int b = threadIdx.x; b < 3 * LW_BINS; b += THREADS) {
    const unsigned long long v = g[b];
    if (v == 0ull) continue;
    g[b] = 0ull;
    const int which = b / LW_BINS, ex = b % LW_BINS;
    const int f1 = (ex ? ex : 1) - 1;  // the importance is m 2^(f - 150): units of 2^-149 and 2^-298
    const int shift = which == 0 ? f1 : (which == 1 ? 2 * f1 + 24 : 2 * f1);
    unsigned long long* digit = which == 0 ? d1 : d2;
    const int d = shift >> 5, r = shift & 31;
    const unsigned long long vl = (v & 0xffffffffull) << r, vh = (v >> 32) << r;  // each below 2^63
    atomicAdd(&digit[d], vl & 0xffffffffull);
    atomicAdd(&digit[d + 1], (vl >> 32) + (vh & 0xffffffffull));
    atomicAdd(&digit[d + 2], vh >> 32);
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  const double S1 = lw_round(d1, D1, -149), S2 = lw_round(d2, D2, -298);
  const double n = static_cast<double>(layers[layer].n);
  const double mean = __ddiv_rn(S1, n);
  const double var = __dsub_rn(__ddiv_rn(S2, n), __dmul_rn(mean, mean));
  const double v = mean > 0.0 ? __ddiv_rn(var, mean) : 0.0;
  const double bv = __dmul_rn(beta, v);
  const double t = v > c_split ? __dadd_rn(alpha, bv) : __dsub_rn(alpha, bv);
  float thr = __double2float_rn(t);
  if (thr == 0.0f) thr = 0.0f;  // -0 -> +0
  thr_bits[j * n_layers + layer] = __float_as_uint(thr);
}


// Threshold mode, last pass: everything that is left of the step in ONE streaming pass over all
// workers, in ascending worker order per element: step (a) for the workers that are not chosen nodes,
// and for the elements of the index set (a bit per element, written by k_thr_write) the ordered sum
// of step (f) and the zeroing of step (g); `update` gets the sum or +0.  No gather: nothing is read
// at scattered addresses.  grid = tiles.
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_thr_fused(const float* __restrict__ grads, float* __restrict__ acc, float* __restrict__ update,
                const Tile* __restrict__ tiles, const uint32_t* __restrict__ set_bits, uint64_t N, int W,
                float momentum, LeaderSet ls) {
  const Tile t = tiles[blockIdx.x];
  const uint64_t lo = t.a, hi = lo + t.len;
  const uint64_t base = lo & ~static_cast<uint64_t>(TILE - 1);
  constexpr int SPT = 2;                          // slots per thread and trip (keeps the kernel at 4 CTAs per SM)
  constexpr int TRIPS = TILE / 4 / THREADS / SPT;  // the tile is walked in two halves
#pragma unroll 1
  for (int trip = 0; trip < TRIPS; ++trip) {
    uint64_t e0[SPT];
    uint32_t in_set[SPT];  // four bits per slot
    float sum[SPT][4];
    bool any = false;
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
      e0[s] = base + static_cast<uint64_t>((trip * SPT + s) * THREADS + threadIdx.x) * 4;
      const bool inside = e0[s] < hi && e0[s] + 4 > lo;
      any = any || inside;
      in_set[s] = inside ? (set_bits[e0[s] >> 5] >> (e0[s] & 31u)) & 0xFu : 0u;
#pragma unroll
      for (int c = 0; c < 4; ++c) sum[s][c] = 0.0f;
    }
    if (!__syncthreads_or(any)) continue;  // this half of the window lies outside a ragged tile
    // the loads of worker w + 1 are issued before worker w's values are combined and stored
    auto chosen = [&](int w) {
      bool c = false;
#pragma unroll
      for (int j = 0; j < MAX_LEADERS; ++j) c = c || (j < ls.n && ls.r[j] == w);
      return c;
    };
    auto fetch = [&](int w, bool is_chosen, float (&gv)[SPT][4], float (&av)[SPT][4]) {
      const float* g = grads + static_cast<uint64_t>(w) * N;
      const float* a = acc + static_cast<uint64_t>(w) * N;
#pragma unroll
      for (int s = 0; s < SPT; ++s) {
        load4_stream<VEC>(a, e0[s], lo, hi, av[s]);
        if (is_chosen) {
#pragma unroll
          for (int c = 0; c < 4; ++c) gv[s][c] = 0.0f;
        } else {
          load4_stream<VEC>(g, e0[s], lo, hi, gv[s]);
        }
      }
    };
    float gv[SPT][4], av[SPT][4];
    bool is_chosen = chosen(0);
    fetch(0, is_chosen, gv, av);
    for (int w = 0; w < W; ++w) {
      float gn[SPT][4], an[SPT][4];
      bool next_chosen = false;
      if (w + 1 < W) {
        next_chosen = chosen(w + 1);
        fetch(w + 1, next_chosen, gn, an);
      }
      float* a = acc + static_cast<uint64_t>(w) * N;
#pragma unroll
      for (int s = 0; s < SPT; ++s) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (!is_chosen) av[s][c] = accumulate(av[s][c], gv[s][c], momentum);
          if ((in_set[s] >> c) & 1u) {
            sum[s][c] = (w == 0) ? av[s][c] : __fadd_rn(sum[s][c], av[s][c]);
            av[s][c] = 0.0f;
          }
        }
        if (!is_chosen || in_set[s]) store4<VEC>(a, e0[s], lo, hi, av[s]);
      }
      if (w + 1 < W) {
#pragma unroll
        for (int s = 0; s < SPT; ++s) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            gv[s][c] = gn[s][c];
            av[s][c] = an[s][c];
          }
        }
        is_chosen = next_chosen;
      }
    }
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
      float out[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) out[c] = ((in_set[s] >> c) & 1u) ? __fadd_rn(0.0f, sum[s][c]) : 0.0f;
      store4<VEC>(update, e0[s], lo, hi, out);
    }
  }
}

// Byte mask of the index set of a threshold-mode step (accessor): grid-stride over the list, whose length
// is only known on the device.
__global__ void __launch_bounds__(THREADS)
    k_thr_mask(const uint32_t* __restrict__ sel_idx, const uint32_t* __restrict__ list_len, uint32_t capacity,
               uint8_t* __restrict__ dst) {
  const uint32_t len = min(*list_len, capacity);
  for (uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x; j < len;
       j += static_cast<uint64_t>(gridDim.x) * THREADS)
    dst[sel_idx[j]] = 1;
}

}  // namespace iwp

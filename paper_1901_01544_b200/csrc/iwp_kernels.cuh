// sm_100a kernels of the importance-weighted pruning step (Algorithm 1 of the paper).
//
// Nothing here is a dense contraction, so there are no tensor-core instructions: every
// kernel is bound by HBM traffic (or, for the small ones, by launch latency).  The work is
// organised so that the W*N residual/gradient stream is touched as few times as possible
// and always with coalesced 128-bit accesses.
//
// IEEE exactness: the residual add, the eps guard and the division use the explicit
// round-to-nearest intrinsics, so the results do not depend on compiler contraction or
// fast-math flags, and denormals are kept.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_plan.hpp"

namespace iwp {

constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int STATUS_INTERNAL = -4;
constexpr int STATUS_CAPACITY = -6;

// radix-select digit plan over the 32-bit importance pattern (bit 31 is always 0)
__host__ __device__ constexpr int pass_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__host__ __device__ constexpr int pass_bins(int pass) { return pass == 2 ? 1024 : 2048; }
constexpr int N_PASSES = 3;

// Per (tiled layer, worker) pair: the threshold guess of the single-read path and what the
// fused accumulate pass found with it.
struct PairInfo {
  uint32_t guess;  // candidates include every element with importance pattern >= guess; GUESS_NONE = none
  uint32_t total;  // number of elements of the layer that reach the guess
  uint32_t flags;  // bit 0: some (tile, worker) slot or staging queue overflowed
  uint32_t gm;     // bit pattern of the pre-test multiplier derived from the guess
};

// The candidates hold the exact top-k iff there are at least k of them and none was dropped.
__device__ __forceinline__ bool pair_is_cand(const PairInfo& pi, uint32_t k) {
  return pi.guess != GUESS_NONE && pi.total >= k && (pi.flags & 1u) == 0u;
}

// Which workers a launch of the select kernels covers: blockIdx.y runs over the covered workers.
//   ALL: every worker;  ONLY: worker a, then worker b (b < 0 or b == a: a alone);
//   EXCEPT: every worker but a and b, ascending.
struct WorkerSel {
  int mode, a, b;
  enum { ALL = 0, ONLY = 1, EXCEPT = 2 };
};
__host__ __device__ inline int sel_count(const WorkerSel& ws, int W) {
  const int named = (ws.b < 0 || ws.b == ws.a) ? 1 : 2;
  return ws.mode == WorkerSel::ALL ? W : (ws.mode == WorkerSel::ONLY ? named : W - named);
}
__device__ __forceinline__ int sel_worker(const WorkerSel& ws, int y) {
  if (ws.mode == WorkerSel::ALL) return y;
  if (ws.mode == WorkerSel::ONLY) return y == 0 ? ws.a : ws.b;
  const int b = ws.b < 0 ? ws.a : ws.b;
  const int lo = ws.a < b ? ws.a : b, hi = ws.a < b ? b : ws.a;
  int w = y;
  if (w >= lo) ++w;
  if (hi != lo && w >= hi) ++w;
  return w;
}

// ---------------------------------------------------------------------------------------
// element helpers
// ---------------------------------------------------------------------------------------

// Algorithm 1, mask line: |grad / w|, with the eps guard; the bit pattern of a non-negative
// float orders like the float, so the unsigned pattern is the sort key.
__device__ __forceinline__ uint32_t imp_key(float acc, float w, float eps) {
  return __float_as_uint(__fdiv_rn(fabsf(acc), __fadd_rn(fabsf(w), eps)));
}

// Step (a) with Eq. 3's momentum on the locally kept residual: one rounded product, one rounded sum
// (m = 1 leaves the residual as it is: plain accumulation).
__device__ __forceinline__ float accumulate(float acc, float g, float m) { return __fadd_rn(__fmul_rn(m, acc), g); }

__device__ __forceinline__ float imp_den(float w, float eps) { return __fadd_rn(fabsf(w), eps); }
__device__ __forceinline__ uint32_t imp_key_den(float acc, float den) {
  return __float_as_uint(__fdiv_rn(fabsf(acc), den));
}

// A slot is four consecutive floats starting at a multiple of four elements.  [lo, hi) is
// the valid flat range; a slot fully inside it is moved with one 128-bit access when VEC.
template <bool VEC>
__device__ __forceinline__ void load4(const float* __restrict__ p, uint64_t e0, uint64_t lo, uint64_t hi,
                                      float (&v)[4]) {
  if (VEC && e0 >= lo && e0 + 4 <= hi) {
    const float4 t = *reinterpret_cast<const float4*>(p + e0);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint64_t e = e0 + c;
      v[c] = (e >= lo && e < hi) ? p[e] : 0.0f;
    }
  }
}

// same, for data that is read exactly once (the gradients): streaming / evict-first
template <bool VEC>
__device__ __forceinline__ void load4_stream(const float* __restrict__ p, uint64_t e0, uint64_t lo, uint64_t hi,
                                             float (&v)[4]) {
  if (VEC && e0 >= lo && e0 + 4 <= hi) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p + e0));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint64_t e = e0 + c;
      v[c] = (e >= lo && e < hi) ? __ldcs(p + e) : 0.0f;
    }
  }
}

template <bool VEC>
__device__ __forceinline__ void store4(float* __restrict__ p, uint64_t e0, uint64_t lo, uint64_t hi,
                                       const float (&v)[4]) {
  if (VEC && e0 >= lo && e0 + 4 <= hi) {
    *reinterpret_cast<float4*>(p + e0) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint64_t e = e0 + c;
      if (e >= lo && e < hi) p[e] = v[c];
    }
  }
}

// ---------------------------------------------------------------------------------------
// block helpers (THREADS = 256)
// ---------------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t x) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, x, d);
    if (lane >= d) x += y;
  }
  return x;
}

// Exclusive prefix sum over the block in thread order; `total` = block sum.
// sh_warp: WARPS words of shared memory.  Contains two __syncthreads().
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t x, uint32_t* sh_warp, uint32_t& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const uint32_t incl = warp_incl_scan(x);
  if (lane == 31) sh_warp[wid] = incl;
  __syncthreads();
  uint32_t woff = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < WARPS; ++i) {
    const uint32_t v = sh_warp[i];
    if (i < wid) woff += v;
    tot += v;
  }
  __syncthreads();
  total = tot;
  return woff + incl - x;
}

// Radix-select digit step on a histogram in shared memory: finds the digit d with
//   count(digit > d) < krem <= count(digit >= d)
// res[0] = d, res[1] = krem - count(digit > d), res[2] = 1 if found.  sh_scan: THREADS words.
template <int NT = THREADS>
__device__ __forceinline__ void find_digit(const uint32_t* hist, int nb, uint32_t krem, uint32_t* sh_scan,
                                           uint32_t* res) {
  const int tid = threadIdx.x;
  const int per = nb / NT;
  uint32_t local = 0;
  for (int b = 0; b < per; ++b) local += hist[tid * per + b];
  sh_scan[tid] = local;
  if (tid == 0) res[2] = 0;
  __syncthreads();
  for (int d = 1; d < NT; d <<= 1) {  // inclusive suffix sum over threads
    const uint32_t v = (tid + d < NT) ? sh_scan[tid + d] : 0u;
    __syncthreads();
    sh_scan[tid] += v;
    __syncthreads();
  }
  const uint32_t incl = sh_scan[tid];
  const uint32_t excl = incl - local;
  if (excl < krem && krem <= incl) {
    uint32_t running = excl;
    for (int b = per - 1; b >= 0; --b) {
      const uint32_t h = hist[tid * per + b];
      if (running + h >= krem) {
        res[0] = static_cast<uint32_t>(tid * per + b);
        res[1] = krem - running;
        res[2] = 1;
        break;
      }
      running += h;
    }
  }
  __syncthreads();
}

// Exact radix select on keys held in shared memory: the krem-th largest of n keys.
// On success T = that key and r = how many T-valued keys belong to the top krem.
// hist: NBINS words, sh_scan: NT words, res: 4 words.  Returns false if the counts are
// inconsistent (krem > n).  All NT threads of the block must call it.
template <int NT = THREADS>
__device__ __forceinline__ bool smem_radix_select(const uint32_t* keys, uint32_t n, uint32_t krem, uint32_t* hist,
                                                  uint32_t* sh_scan, uint32_t* res, uint32_t& T, uint32_t& r) {
  const int tid = threadIdx.x;
  uint32_t prefix = 0;
#pragma unroll 1
  for (int pass = 0; pass < N_PASSES; ++pass) {
    const int shift = pass_shift(pass), nb = pass_bins(pass);
    const int prev_shift = pass == 0 ? 31 : pass_shift(pass - 1);
    const uint32_t want = prefix >> prev_shift;
    for (int b = tid; b < nb; b += NT) hist[b] = 0;
    __syncthreads();
    for (uint32_t i = tid; i < n; i += NT) {
      const uint32_t key = keys[i];
      if ((key >> prev_shift) == want) atomicAdd(&hist[(key >> shift) & (nb - 1)], 1u);
    }
    __syncthreads();
    find_digit<NT>(hist, nb, krem, sh_scan, res);
    const bool found = res[2] != 0;
    const uint32_t d = res[0], kr = res[1];
    __syncthreads();
    if (!found) return false;
    prefix |= d << shift;
    krem = kr;
  }
  T = prefix;
  r = krem;
  return true;
}

// Warp-aggregated increment of a shared-memory histogram: lanes that hit the same bin
// elect one lane that adds the whole group's count.  Must be called by all 32 lanes.
__device__ __forceinline__ void hist_add_aggregated(uint32_t* hist, bool valid, uint32_t bin) {
  const uint32_t tag = valid ? bin : 0xffffffffu;
  const uint32_t peers = __match_any_sync(0xffffffffu, tag);
  const int lane = threadIdx.x & 31;
  if (valid && (__ffs(peers) - 1) == lane) atomicAdd(&hist[bin], static_cast<uint32_t>(__popc(peers)));
}

// ---------------------------------------------------------------------------------------
// tiled path, step (a) alone: residual accumulation  acc += grads, and update <- 0.
// Used when speculation is off.  grid = tiles; each CTA walks the W workers of one tile.
// ---------------------------------------------------------------------------------------
template <bool VEC>
__global__ void __launch_bounds__(THREADS) k_accumulate(const float* __restrict__ grads, float* __restrict__ acc,
                                                         float* __restrict__ update, const Tile* __restrict__ tiles,
                                                         uint64_t N, int W, float momentum) {
  const Tile t = tiles[blockIdx.x];
  const uint64_t lo = t.a, hi = lo + t.len;
  const uint64_t base = lo & ~static_cast<uint64_t>(TILE - 1);
  constexpr int SPT = TILE / 4 / THREADS;  // slots per thread
  uint64_t e0[SPT];
#pragma unroll
  for (int s = 0; s < SPT; ++s) e0[s] = base + static_cast<uint64_t>(s * THREADS + threadIdx.x) * 4;
  const float zero[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int s = 0; s < SPT; ++s) store4<VEC>(update, e0[s], lo, hi, zero);
  for (int w = 0; w < W; ++w) {
    const float* g = grads + static_cast<uint64_t>(w) * N;
    float* a = acc + static_cast<uint64_t>(w) * N;
    float gv[SPT][4], av[SPT][4];
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
      load4_stream<VEC>(g, e0[s], lo, hi, gv[s]);
      load4<VEC>(a, e0[s], lo, hi, av[s]);
    }
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
#pragma unroll
      for (int c = 0; c < 4; ++c) av[s][c] = accumulate(av[s][c], gv[s][c], momentum);
      store4<VEC>(a, e0[s], lo, hi, av[s]);
    }
  }
}

// ---------------------------------------------------------------------------------------
// single-read path, threshold guess: one CTA per (tiled layer, worker) pair evaluates the
// importance the step WILL produce (acc + grad) on a strided, jittered sample of the layer and
// takes the rho-th largest as the guess.  Only a guess: the select stays exact whatever it is.
// grid = pairs; dynamic shared memory = 4 * max sample bytes.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float pretest_multiplier(uint32_t guess, float eps);

// Lazy zeroing of sent residuals (step (g)): instead of scattering W * K four-byte zeros, the
// reduction marks each sent element in a bit mask and the NEXT streaming pass, which reads every
// residual anyway, takes a marked residual as +0.  Layout: one 16-bit field per (512-element
// segment of the flat element space, lane), bit 4 * round + component - exactly the sixteen
// elements a lane of the streaming pass owns - two fields per 32-bit word.
__device__ __forceinline__ uint64_t zmask_word(uint64_t i) { return ((i >> 9) * 32 + ((i & 127) >> 2)) >> 1; }
__device__ __forceinline__ uint32_t zmask_bit(uint64_t i) {
  return 1u << ((((i & 127) >> 2) & 1) * 16 + ((i >> 7) & 3) * 4 + (i & 3));
}
__device__ __forceinline__ bool zmask_test(const uint32_t* __restrict__ zmask, uint64_t i) {
  return (zmask[zmask_word(i)] & zmask_bit(i)) != 0u;
}

__device__ __forceinline__ uint32_t hash32(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
  return x;
}

constexpr int SAMPLE_THREADS = 1024;

__global__ void __launch_bounds__(SAMPLE_THREADS)
    k_sample(const float* __restrict__ grads, const float* __restrict__ weights, const float* __restrict__ acc,
             const LayerDesc* __restrict__ layers, const uint32_t* __restrict__ large_ids, PairInfo* __restrict__ info,
             uint2* __restrict__ guess_tab, const uint32_t* __restrict__ zmask, float eps, uint64_t N, int W,
             uint32_t step, float momentum) {
  extern __shared__ uint32_t keys[];
  __shared__ uint32_t hist[NBINS];
  __shared__ uint32_t sh_scan[SAMPLE_THREADS];
  __shared__ uint32_t res[4];
  const uint32_t pair = blockIdx.x;
  const LayerDesc L = layers[large_ids[pair / W]];
  const int w = pair % W;
  const uint32_t s = L.sample;
  if (s == 0) {
    if (threadIdx.x == 0) {
      const uint32_t gm = __float_as_uint(pretest_multiplier(GUESS_NONE, eps));
      info[pair] = PairInfo{GUESS_NONE, 0u, 0u, gm};
      guess_tab[pair] = make_uint2(GUESS_NONE, gm);
    }
    return;
  }
  const uint32_t groups = s >> 3;
  const uint32_t stride = L.n / groups;  // >= 128 because s <= n / 16
  const float* a = acc + static_cast<uint64_t>(w) * N + L.off;
  const float* g = grads + static_cast<uint64_t>(w) * N + L.off;
  const float* wt = weights + L.off;
  // eight samples per thread and trip, all loads issued before any use (memory-level parallelism)
  for (uint32_t i0 = 0; i0 < s; i0 += SAMPLE_THREADS * 8) {
    float av[8], gv[8], wv[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint32_t i = i0 + u * SAMPLE_THREADS + threadIdx.x;
      av[u] = gv[u] = 0.f;
      wv[u] = 1.f;
      if (i < s) {
        const uint32_t grp = i >> 3;
        const uint32_t jit = hash32(step * 0x9E3779B9u + pair * 0x85EBCA6Bu + grp * 0xC2B2AE35u + 1u) % (stride - 7u);
        const uint32_t pos = grp * stride + jit + (i & 7u);
        const float av_raw = a[pos];
        const bool sent = zmask_test(zmask, static_cast<uint64_t>(L.off) + pos);  // sent last step: counts as +0
        av[u] = sent ? 0.0f : av_raw;
        gv[u] = g[pos];
        wv[u] = wt[pos];
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint32_t i = i0 + u * SAMPLE_THREADS + threadIdx.x;
      if (i < s) keys[i] = imp_key(accumulate(av[u], gv[u], momentum), wv[u], eps);
    }
  }
  __syncthreads();
  uint32_t T, r;
  const bool ok = smem_radix_select<SAMPLE_THREADS>(keys, s, L.rho, hist, sh_scan, res, T, r);
  if (threadIdx.x == 0) {
    // no speculation on a guess whose first radix digit is zero (importance below 2^-126 * 2^-... ): the
    // select's shortcuts for candidates assume that key 0 and digit 0 never belong to a candidate
    const uint32_t guess = (ok && (T >> pass_shift(0)) != 0u) ? T : GUESS_NONE;
    const uint32_t gm = __float_as_uint(pretest_multiplier(guess, eps));
    info[pair] = PairInfo{guess, 0u, 0u, gm};
    guess_tab[pair] = make_uint2(guess, gm);  // read-only copy for the streaming pass (no atomics land on it)
  }
}

// ---------------------------------------------------------------------------------------
// single-read path: steps (a)+(b) fused with candidate emission and with the gather of step (e).
//
// acc += grads, update <- 0, importance of every element; every element whose importance reaches
// its pair's guess is appended, in index order, to the (tile, worker) candidate slot; and every
// worker's accumulated value at the positions of the LEADER's candidates is written to a side
// buffer, so that after the select the reduction reads those few values instead of gathering
// W * K scattered residuals (each of which costs a 128-byte DRAM fetch).
//
// One WARP owns one (tile, worker) pair and walks the tile front to back, 512 elements per
// iteration (four rounds of 32 lanes x one 128-bit slot): candidate order is (iteration, round,
// lane, component) = index order, a running count in a register is all the state, warps never
// wait for each other.  The kernel runs twice per step: first for the leader alone (LEADER =
// true: it also zeroes `update` and records, per segment and lane, its staged mask and ranks),
// then for all other workers, which read that record to place their values in the side buffer.
//
// Cheap pre-test before the exact quotient: with gm = guess * (1 - 2^-20) every element whose
// correctly rounded quotient |acc| / den reaches the guess passes |acc| >= gm * den (the two
// roundings of gm * den and the one of the quotient are each below 2^-23 relative).  Elements that
// pass are staged, in index order, in a per-warp queue in shared memory; the lanes then take one
// entry each, form the exact quotient (one division per lane, not per element), count how many
// really reach the guess, and append ALL staged entries with coalesced stores.  Keeping the few
// entries that fall just short of the guess is harmless: whenever at least k elements of the layer
// reach the guess, the k best of this superset are the k best of the layer.  The argument needs
// normal products, so the pre-test is disabled (gm = 0: everything passes) for tiny guesses or eps.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float pretest_multiplier(uint32_t guess, float eps) {
  if (guess == GUESS_NONE) return __int_as_float(0x7f800000);  // +inf: nothing passes
  const float gf = __uint_as_float(guess);
  const float tiny = 8.673617379884035e-19f;  // 2^-60
  if (!(gf >= tiny) || !(eps >= tiny)) return 0.0f;
  return __fmul_rd(gf, 1.0f - 9.5367431640625e-07f);
}

constexpr int EMIT_QUEUE = 128;  // staged entries per warp and iteration; more than this = overflow

// Candidate entries are re-read several times by the select right after the streaming pass: store
// them with an L2 evict-last policy so that the 6 GB that stream through L2 meanwhile do not push
// them out.
__device__ __forceinline__ uint64_t l2_evict_last_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_keep_u32(uint32_t* ptr, uint32_t v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.u32 [%0], %1, %2;" ::"l"(ptr), "r"(v), "l"(policy) : "memory");
}
__device__ __forceinline__ void st_keep_f32(float* ptr, float v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(ptr), "f"(v), "l"(policy) : "memory");
}
__device__ __forceinline__ void st_keep_u16(uint16_t* ptr, uint16_t v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.u16 [%0], %1, %2;" ::"l"(ptr), "h"(v), "l"(policy) : "memory");
}

// Position, inside one iteration, of the staged element with mask bit b = 4 * round + component:
// the staged elements of earlier rounds, of earlier lanes in the same round, and of earlier
// components of the same lane and round.  `ex` / `tt`: per-round exclusive lane prefix / totals,
// packed 8 bits per round.
__device__ __forceinline__ uint32_t staged_position(uint32_t mask, uint32_t ex, uint32_t tt, uint32_t b) {
  const uint32_t sh = (b >> 2) * 8;
  const uint32_t rounds_before = ((tt * 0x01010100u) >> sh) & 0xFFu;  // byte r of tt * 0x01010100 = sum of rounds < r
  return rounds_before + ((ex >> sh) & 0xFFu) + __popc((mask >> (b & ~3u)) & ((1u << (b & 3u)) - 1u));
}

template <bool VEC, bool LEADER>
__global__ void __launch_bounds__(THREADS, 3)
    k_stream(const float* __restrict__ grads, const float* __restrict__ weights, float* __restrict__ acc,
             float* __restrict__ update, const Tile* __restrict__ tiles, PairInfo* __restrict__ info,
             const uint2* __restrict__ guess_tab, uint32_t* __restrict__ cand_key, float* __restrict__ cand_val,
             uint16_t* __restrict__ cand_idx, uint32_t* __restrict__ cand_cnt, float* __restrict__ side_val,
             uint2* __restrict__ lead_lane, uint32_t* __restrict__ lead_tot, const uint32_t* __restrict__ zmask,
             float eps, uint64_t N, int W, int leader, uint32_t n_tiles, int worker_groups, float momentum) {
  constexpr int ROUNDS = SEG_ELEMS / 128;  // 128-bit slots per lane and iteration = 4
  __shared__ float q_val[WARPS][EMIT_QUEUE];
  __shared__ float q_den[WARPS][EMIT_QUEUE];
  __shared__ uint16_t q_loc[WARPS][EMIT_QUEUE];
  __shared__ __align__(16) float r_val[WARPS][SEG_ELEMS];  // results of the iteration, for run-time indexing
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t tile_id;
  int w;
  if (LEADER) {  // eight tiles of the leader per CTA
    tile_id = blockIdx.x * WARPS + warp;
    w = leader;
    if (tile_id >= n_tiles) return;
  } else {  // up to eight of the other workers of one tile per CTA: the tile's weights come through L1
    tile_id = blockIdx.x / worker_groups;
    const int wi = static_cast<int>(blockIdx.x % worker_groups) * static_cast<int>(blockDim.x >> 5) + warp;
    if (wi >= W - 1) return;
    w = wi < leader ? wi : wi + 1;
  }
  const Tile t = tiles[tile_id];
  const uint64_t lo = t.a, hi = lo + t.len;
  const uint64_t base = lo & ~static_cast<uint64_t>(TILE - 1);
  const bool full = VEC && t.len == TILE;  // every slot of the window is inside the tile
  const uint32_t pair = t.large_index * W + w;
  const uint2 pg = guess_tab[pair];
  const uint32_t guess = pg.x;
  const float gm = __uint_as_float(pg.y);
  const float gme = __fmul_rn(gm, eps);
  const float* g = grads + static_cast<uint64_t>(w) * N;
  float* a = acc + static_cast<uint64_t>(w) * N;
  const uint64_t slot = (static_cast<uint64_t>(tile_id) * W + w) * CAND_CAP;
  const float zero[4] = {0.f, 0.f, 0.f, 0.f};
  float* qv = q_val[warp];
  float* qd = q_den[warp];
  uint16_t* ql = q_loc[warp];
  float* res = r_val[warp] + lane * 4;
  uint32_t count = 0;    // entries appended to the slot so far (the same in every lane)
  uint32_t reached = 0;  // of those, how many reach the guess exactly
  bool overflow = false;
  const uint64_t keep = l2_evict_last_policy();
  // The tile covers the segments it0 .. it1 of its window.  The loads of segment it + 1 are issued
  // as soon as the arithmetic of segment it is done, so they are in flight while the rare-path work
  // of segment it (side values, staging, exact quotients) runs out of shared memory.
  const uint32_t it0 = static_cast<uint32_t>((lo - base) / SEG_ELEMS);
  const uint32_t it1 = static_cast<uint32_t>((hi - 1 - base) / SEG_ELEMS);
  float gv[ROUNDS][4], av[ROUNDS][4], den[ROUNDS][4];
  uint32_t zm_next = 0;
  uint2 ll_next = make_uint2(0u, 0u);
  uint32_t lt_next = 0;
  auto fetch = [&](uint32_t it) {
    const uint64_t seg = base + it * SEG_ELEMS;
    const uint64_t first = seg + static_cast<uint64_t>(lane) * 4;
    // residuals sent in the previous step count as +0 (they are overwritten either way)
    zm_next = reinterpret_cast<const uint16_t*>(zmask)[(seg >> 9) * 32 + lane];
    if (!LEADER) {  // the leader's record for this segment: (mask | count << 16, lane prefix), round totals
      const uint64_t sigma = static_cast<uint64_t>(tile_id) * SEGS_PER_TILE + it;
      ll_next = lead_lane[sigma * 32 + lane];
      lt_next = lead_tot[sigma];
    }
    if (full) {
      const float4* g4 = reinterpret_cast<const float4*>(g + first);
      const float4* a4 = reinterpret_cast<const float4*>(a + first);
      const float4* w4 = reinterpret_cast<const float4*>(weights + first);
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) {
        const float4 x = __ldcs(g4 + s * 32), y = __ldcs(a4 + s * 32), z = w4[s * 32];
        gv[s][0] = x.x; gv[s][1] = x.y; gv[s][2] = x.z; gv[s][3] = x.w;
        av[s][0] = y.x; av[s][1] = y.y; av[s][2] = y.z; av[s][3] = y.w;
        den[s][0] = z.x; den[s][1] = z.y; den[s][2] = z.z; den[s][3] = z.w;
      }
    } else {
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) {
        const uint64_t e0 = first + s * 128;
        load4_stream<VEC>(g, e0, lo, hi, gv[s]);
        load4_stream<VEC>(a, e0, lo, hi, av[s]);
        load4<VEC>(weights, e0, lo, hi, den[s]);
      }
    }
  };
  fetch(it0);
#pragma unroll 1
  for (uint32_t it = it0; it <= it1; ++it) {
    const uint64_t seg = base + it * SEG_ELEMS;
    const uint64_t first = seg + static_cast<uint64_t>(lane) * 4;  // this lane's slot in round 0
    const uint64_t sigma = static_cast<uint64_t>(tile_id) * SEGS_PER_TILE + it;  // global segment id
    const uint32_t zm = zm_next;
    const uint2 ll = ll_next;
    const uint32_t lt = lt_next;
    uint32_t inrange = 0xFFFFu;
    if (!full) {
      inrange = 0;
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint64_t e = first + s * 128 + c;
          inrange |= (e >= lo && e < hi) ? (1u << (4 * s + c)) : 0u;
        }
      }
    }
    if (zm) {
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) {
#pragma unroll
        for (int c = 0; c < 4; ++c) av[s][c] = ((zm >> (4 * s + c)) & 1u) ? 0.0f : av[s][c];
      }
    }
    uint32_t m = 0;  // bit (4 s + c): passes the pre-test
#pragma unroll
    for (int s = 0; s < ROUNDS; ++s) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        av[s][c] = accumulate(av[s][c], gv[s][c], momentum);
        // gm * (|w| + eps) in one fused operation; its rounding differs from the exact denominator's
        // by parts in 2^24, far inside the 2^-20 slack of gm (den[][] holds the raw weights here)
        m |= (fabsf(av[s][c]) >= __fmaf_rn(gm, fabsf(den[s][c]), gme)) ? (1u << (4 * s + c)) : 0u;
      }
    }
    // results: to HBM, and into shared memory so that the rare-path loops below can pick single
    // elements by a run-time index without keeping all sixteen in registers
#pragma unroll
    for (int s = 0; s < ROUNDS; ++s)
      *reinterpret_cast<float4*>(res + s * 128) = make_float4(av[s][0], av[s][1], av[s][2], av[s][3]);
    if (full) {
      float4* a4 = reinterpret_cast<float4*>(a + first);
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) __stcs(a4 + s * 32, make_float4(av[s][0], av[s][1], av[s][2], av[s][3]));
      if (LEADER) {
        float4* u4 = reinterpret_cast<float4*>(update + first);
#pragma unroll
        for (int s = 0; s < ROUNDS; ++s) __stcs(u4 + s * 32, make_float4(0.f, 0.f, 0.f, 0.f));
      }
    } else {
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) {
        store4<VEC>(a, first + s * 128, lo, hi, av[s]);
        if (LEADER) store4<VEC>(update, first + s * 128, lo, hi, zero);
      }
    }
    m &= inrange;
    if (it < it1) fetch(it + 1);  // in flight during the rare-path work below

    if (!LEADER) {  // this worker's value at every position of the leader's slot (step (e) without a gather)
      const uint32_t mL = ll.x & 0xFFFFu, countL = ll.x >> 16;
      for (uint32_t mm = mL; mm; mm &= mm - 1) {
        const uint32_t b = __ffs(mm) - 1;
        const uint32_t pos = countL + staged_position(mL, ll.y, lt, b);
        if (pos < CAND_CAP) st_keep_f32(side_val + slot + pos, res[(b >> 2) * 128 + (b & 3u)], keep);
      }
    }

    const bool any = __any_sync(0xffffffffu, m != 0u);
    uint32_t excl = 0, tot = 0;
    if (any) {  // queue position in index order: per-round counts packed 8 bits each (<= 128 per round)
      uint32_t packed = 0;
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) packed |= static_cast<uint32_t>(__popc((m >> (4 * s)) & 0xFu)) << (8 * s);
      const uint32_t incl = warp_incl_scan(packed);
      tot = __shfl_sync(0xffffffffu, incl, 31);
      excl = incl - packed;
    }
    if (LEADER) {
      lead_lane[sigma * 32 + lane] = make_uint2(m | (count << 16), excl);
      if (lane == 0) lead_tot[sigma] = tot;
    }
    if (any) {
      for (uint32_t mm = m; mm; mm &= mm - 1) {
        const uint32_t b = __ffs(mm) - 1;
        const uint32_t pos = staged_position(m, excl, tot, b);
        if (pos < EMIT_QUEUE) {
          const uint32_t off = (b >> 2) * 128 + (b & 3u);
          qv[pos] = res[off];
          qd[pos] = imp_den(weights[first + off], eps);  // re-read through L1: only staged elements get here
          ql[pos] = static_cast<uint16_t>(static_cast<uint32_t>(first - base) + off);
        }
      }
      uint32_t nq = (tot & 0xFFu) + ((tot >> 8) & 0xFFu) + ((tot >> 16) & 0xFFu) + (tot >> 24);
      if (nq > EMIT_QUEUE) {
        overflow = true;
        nq = EMIT_QUEUE;
      }
      __syncwarp();
      for (uint32_t j0 = 0; j0 < nq; j0 += 32) {
        const uint32_t j = j0 + lane;
        bool hit = false;
        if (j < nq) {
          const float v = qv[j];
          const uint32_t key = imp_key_den(v, qd[j]);  // Algorithm 1's |grad / w|, exactly rounded
          hit = key >= guess;
          const uint32_t pos = count + j;
          if (pos < CAND_CAP) {
            st_keep_u32(cand_key + slot + pos, key, keep);
            st_keep_f32(cand_val + slot + pos, v, keep);
            st_keep_u16(cand_idx + slot + pos, ql[j], keep);
          }
        }
        reached += __popc(__ballot_sync(0xffffffffu, hit));
      }
      count += nq;
      __syncwarp();
    }
  }
  // pad the slot to a multiple of four entries with key 0, so that readers can take whole 128-bit
  // groups without testing every entry (no candidate has key 0: a zero guess is never used)
  {
    const uint32_t stored = count < CAND_CAP ? count : CAND_CAP;
    const uint32_t pad_at = stored + lane;
    if (pad_at < ((stored + 3u) & ~3u)) st_keep_u32(cand_key + slot + pad_at, 0u, keep);
  }
  if (lane == 0) {
    st_keep_u32(cand_cnt + static_cast<uint64_t>(tile_id) * W + w, count, keep);
    if (reached) atomicAdd(&info[pair].total, reached);
    if (overflow || count > CAND_CAP) atomicOr(&info[pair].flags, 1u);
  }
}

// The candidates of (chunk, worker): warp q takes the chunk's tiles 16 q .. 16 q + 15 (consecutive,
// so that warp order is index order), four tiles at a time; each lane reads entries 4 lane .. 4 lane + 3
// of a slot with one 128-bit load (a slot rarely holds more than 128 entries; a tail loop covers the
// rest) and all loads of a batch are issued before any is used.  `f(key)` sees every stored candidate,
// and in addition some keys 0 (padding, slots shorter than 128 entries), which `f` must ignore - every
// use below does so by construction, because a candidate's key and first digit are never 0.
constexpr uint32_t TILES_PER_WARP = CHUNK_TILES / WARPS;

template <typename F>
__device__ __forceinline__ void for_each_candidate(const Chunk& c, int w, int W, const uint32_t* __restrict__ cand_cnt,
                                                   const uint32_t* __restrict__ cand_key, F&& f) {
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t t_begin = warp * TILES_PER_WARP;
  const uint32_t t_end = min(c.n_tiles, t_begin + TILES_PER_WARP);
  for (uint32_t tb = t_begin; tb < t_end; tb += 4) {
    uint32_t cnt[4];
    uint4 k4[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      cnt[q] = (tb + q < t_end) ? min(cand_cnt[static_cast<uint64_t>(c.first_tile + tb + q) * W + w], CAND_CAP) : 0u;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4* kp = reinterpret_cast<const uint4*>(cand_key + (static_cast<uint64_t>(c.first_tile + tb + q) * W + w) * CAND_CAP);
      k4[q] = (lane * 4 < cnt[q]) ? kp[lane] : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {  // groups past the count were not loaded (zeros); the last group is zero-padded
      f(k4[q].x);
      f(k4[q].y);
      f(k4[q].z);
      f(k4[q].w);
      if (cnt[q] > 128) {
        const uint4* kp = reinterpret_cast<const uint4*>(cand_key + (static_cast<uint64_t>(c.first_tile + tb + q) * W + w) * CAND_CAP);
        for (uint32_t j0 = 128; j0 < cnt[q]; j0 += 128) {
          const uint32_t j = j0 + lane * 4;
          if (j < cnt[q]) {
            const uint4 k = kp[j >> 2];
            f(k.x);
            f(k.y);
            f(k.z);
            f(k.w);
          }
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// tiled path, step (c): exact radix select of the k-th largest key per (worker, layer).
// Every kernel below serves both kinds of pair: those whose candidates hold the top-k read the
// candidate slots, the others read the residual and the weights again (multi-pass exact path).
// ---------------------------------------------------------------------------------------

// One histogram pass over a chunk: keys that match the prefix found so far are counted by
// their next digit.  grid = (chunks, W).  In the last pass every CTA additionally leaves, per chunk,
// the number of keys above the prefix and the suffix sums of its low-digit histogram; with the
// threshold known, the compaction derives every chunk's (#keys > T, #keys == T) from those without
// another look at the keys (chunk_sfx == nullptr: skipped, a counting kernel runs instead).
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_hist(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
           const LayerDesc* __restrict__ layers, const PairInfo* __restrict__ info,
           const uint32_t* __restrict__ cand_key, const uint32_t* __restrict__ cand_cnt,
           const uint2* __restrict__ state,
           uint32_t* __restrict__ hist, uint32_t* __restrict__ chunk_sfx, uint2* __restrict__ chunk_cnt, float eps,
           uint64_t N, int W, int pass, uint32_t n_chunks, WorkerSel ws) {
  __shared__ uint32_t sh[NBINS];
  __shared__ uint32_t sh_warp[WARPS];
  __shared__ uint32_t sh_above;
  const Chunk c = chunks[blockIdx.x];
  const int w = sel_worker(ws, static_cast<int>(blockIdx.y));
  const LayerDesc L = layers[c.layer];
  const uint32_t pair = static_cast<uint32_t>(L.large_index) * W + w;
  const int shift = pass_shift(pass), nb = pass_bins(pass);
  const int prev_shift = pass == 0 ? 31 : pass_shift(pass - 1);
  const uint2 st_in = pass == 0 ? make_uint2(0u, L.k) : state[pair];
  const uint32_t want = pass == 0 ? 0u : (st_in.x >> prev_shift);
  const bool last_pass = pass == N_PASSES - 1;
  for (int b = threadIdx.x; b < nb; b += THREADS) sh[b] = 0;
  if (threadIdx.x == 0) sh_above = 0;
  __syncthreads();
  uint32_t above = 0;  // keys whose higher digits already exceed the prefix (needed in the last pass only)
  const PairInfo pi = info[pair];
  if (pair_is_cand(pi, L.k) && pass == 0) {
    // Every candidate is at or just above the guess, so almost all of them fall into the guess's own
    // first-digit bin or the next two: count those in registers (one shared-memory atomic per lane
    // would serialise on three addresses) and leave only the rest to atomics.
    const uint32_t g0 = pi.guess >> shift;
    uint32_t c0 = 0, c1 = 0, c2 = 0;
    for_each_candidate(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      const uint32_t d = (key >> shift) - g0;
      c0 += d == 0u ? 1u : 0u;
      c1 += d == 1u ? 1u : 0u;
      c2 += d == 2u ? 1u : 0u;
      if (d > 2u && key != 0u) atomicAdd(&sh[(key >> shift) & (nb - 1)], 1u);
    });
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      c0 += __shfl_xor_sync(0xffffffffu, c0, d);
      c1 += __shfl_xor_sync(0xffffffffu, c1, d);
      c2 += __shfl_xor_sync(0xffffffffu, c2, d);
    }
    if ((threadIdx.x & 31) == 0) {
      if (c0) atomicAdd(&sh[g0 & (nb - 1)], c0);
      if (c1) atomicAdd(&sh[(g0 + 1) & (nb - 1)], c1);
      if (c2) atomicAdd(&sh[(g0 + 2) & (nb - 1)], c2);
    }
  } else if (pair_is_cand(pi, L.k)) {
    for_each_candidate(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      const uint32_t hi_part = key >> prev_shift;
      if (hi_part == want) atomicAdd(&sh[(key >> shift) & (nb - 1)], 1u);
      above += hi_part > want ? 1u : 0u;
    });
  } else {
    const uint64_t lo = c.a, hi = lo + c.len;
    const uint64_t s0 = lo & ~3ull;
    const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
    const float* a = acc + static_cast<uint64_t>(w) * N;
    for (uint32_t it = 0; it < n_iter; ++it) {
      const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
      float av[4], wv[4];
      load4<VEC>(a, e0, lo, hi, av);
      load4<VEC>(weights, e0, lo, hi, wv);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t e = e0 + q;
        const uint32_t key = imp_key(av[q], wv[q], eps);
        const bool in = e >= lo && e < hi;
        const bool valid = in && (key >> prev_shift) == want;  // pass 0: bit 31 is 0 == want
        hist_add_aggregated(sh, valid, (key >> shift) & (nb - 1));
        above += (in && (key >> prev_shift) > want) ? 1u : 0u;
      }
    }
  }
  if (last_pass && chunk_sfx != nullptr) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xffffffffu, above, d);
    if ((threadIdx.x & 31) == 0 && above) atomicAdd(&sh_above, above);
  }
  __syncthreads();
  uint32_t* gh = hist + static_cast<uint64_t>(pair) * NBINS;
  for (int b = threadIdx.x; b < nb; b += THREADS) {
    const uint32_t v = sh[b];
    if (v) atomicAdd(&gh[b], v);
  }
  if (last_pass && chunk_sfx != nullptr) {  // suffix sums S[b] = sum of this chunk's bins >= b, and the count above the prefix
    static_assert(pass_bins(N_PASSES - 1) == THREADS * 4, "four bins per thread in the last pass");
    const uint32_t h0 = sh[threadIdx.x * 4], h1 = sh[threadIdx.x * 4 + 1], h2 = sh[threadIdx.x * 4 + 2],
                   h3 = sh[threadIdx.x * 4 + 3];
    uint32_t total;
    const uint32_t before = block_excl_scan(h0 + h1 + h2 + h3, sh_warp, total);
    const uint32_t s0 = total - before;
    uint4 sfx = make_uint4(s0, s0 - h0, s0 - h0 - h1, s0 - h0 - h1 - h2);
    uint32_t* dst = chunk_sfx + (static_cast<uint64_t>(w) * n_chunks + blockIdx.x) * pass_bins(N_PASSES - 1);
    reinterpret_cast<uint4*>(dst)[threadIdx.x] = sfx;
    if (threadIdx.x == 0) chunk_cnt[static_cast<uint64_t>(w) * n_chunks + blockIdx.x] = make_uint2(sh_above, 0u);
  }
}

// Digit decision for (worker, layer) pairs of the tiled path; grid = (tiled layers, covered workers).
// Reads the pair's histogram, clears it for the next pass, extends the key prefix.
// After the last pass state = (threshold key T, number r of T-valued elements to keep).
__global__ void __launch_bounds__(THREADS)
    k_find_digit(uint2* __restrict__ state, uint32_t* __restrict__ hist, const LayerDesc* __restrict__ layers,
                 const uint32_t* __restrict__ large_ids, int* __restrict__ status, int W, int pass,
                 WorkerSel ws) {
  __shared__ uint32_t sh[NBINS];
  __shared__ uint32_t sh_scan[THREADS];
  __shared__ uint32_t res[4];
  const uint32_t pair = blockIdx.x * static_cast<uint32_t>(W) + static_cast<uint32_t>(sel_worker(ws, static_cast<int>(blockIdx.y)));
  const int nb = pass_bins(pass), shift = pass_shift(pass);
  uint32_t* gh = hist + static_cast<uint64_t>(pair) * NBINS;
  for (int b = threadIdx.x; b < nb; b += THREADS) {
    sh[b] = gh[b];
    gh[b] = 0;
  }
  __syncthreads();
  uint32_t prefix, krem;
  if (pass == 0) {
    prefix = 0;
    krem = layers[large_ids[pair / W]].k;
  } else {
    const uint2 s = state[pair];
    prefix = s.x;
    krem = s.y;
  }
  find_digit(sh, nb, krem, sh_scan, res);
  if (threadIdx.x == 0) {
    if (res[2]) {
      state[pair] = make_uint2(prefix | (res[0] << shift), res[1]);
    } else {
      atomicMin(status, STATUS_INTERNAL);
      state[pair] = make_uint2(0xffffffffu, 0u);  // selects nothing
    }
  }
}

// Per chunk: how many keys are above the threshold and how many equal it.  grid = (chunks, W).
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_count(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
            const LayerDesc* __restrict__ layers, const PairInfo* __restrict__ info,
            const uint32_t* __restrict__ cand_key, const uint32_t* __restrict__ cand_cnt, const uint2* __restrict__ state,
            uint2* __restrict__ chunk_cnt, float eps, uint64_t N, int W, uint32_t n_chunks) {
  __shared__ uint32_t sh_cnt[2];
  const Chunk c = chunks[blockIdx.x];
  const int w = blockIdx.y;
  const LayerDesc L = layers[c.layer];
  const uint32_t pair = static_cast<uint32_t>(L.large_index) * W + w;
  const uint32_t T = state[pair].x;
  if (threadIdx.x < 2) sh_cnt[threadIdx.x] = 0;
  __syncthreads();
  uint32_t gt = 0, eq = 0;
  if (pair_is_cand(info[pair], L.k)) {
    for_each_candidate(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      gt += key > T ? 1u : 0u;
      eq += key == T ? 1u : 0u;
    });
  } else {
    const uint64_t lo = c.a, hi = lo + c.len;
    const uint64_t s0 = lo & ~3ull;
    const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
    const float* a = acc + static_cast<uint64_t>(w) * N;
    for (uint32_t it = 0; it < n_iter; ++it) {
      const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
      float av[4], wv[4];
      load4<VEC>(a, e0, lo, hi, av);
      load4<VEC>(weights, e0, lo, hi, wv);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t e = e0 + q;
        const bool in = e >= lo && e < hi;
        const uint32_t key = imp_key(av[q], wv[q], eps);
        gt += (in && key > T) ? 1u : 0u;
        eq += (in && key == T) ? 1u : 0u;
      }
    }
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    gt += __shfl_xor_sync(0xffffffffu, gt, d);
    eq += __shfl_xor_sync(0xffffffffu, eq, d);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&sh_cnt[0], gt);
    atomicAdd(&sh_cnt[1], eq);
  }
  __syncthreads();
  if (threadIdx.x == 0) chunk_cnt[static_cast<uint64_t>(w) * n_chunks + blockIdx.x] = make_uint2(sh_cnt[0], sh_cnt[1]);
}

// Step (d): stable compaction of the selected elements of a chunk into the worker's list.
// An element is selected if key > T, or key == T and fewer than r T-valued elements of the
// layer precede it; its list position is (#greater before it) + min(#equal before it, r).
// grid = (chunks, W).
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_write(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
            const Tile* __restrict__ tiles, const LayerDesc* __restrict__ layers, const PairInfo* __restrict__ info,
            const uint32_t* __restrict__ cand_key, const float* __restrict__ cand_val,
            const uint16_t* __restrict__ cand_idx, const uint32_t* __restrict__ cand_cnt,
            const uint2* __restrict__ state, const uint2* __restrict__ chunk_cnt, uint32_t* __restrict__ sel_idx,
            float* __restrict__ sel_val, uint32_t* __restrict__ sel_slot, const uint32_t* __restrict__ chunk_sfx,
            int* __restrict__ status, float eps, uint64_t N, uint64_t K, int W, uint32_t n_chunks, int leader,
            WorkerSel ws) {
  __shared__ uint32_t sh_warp[WARPS];
  __shared__ uint32_t sh_base[2];
  const Chunk c = chunks[blockIdx.x];
  const int w = sel_worker(ws, static_cast<int>(blockIdx.y));
  const LayerDesc L = layers[c.layer];
  const uint32_t pair = static_cast<uint32_t>(L.large_index) * W + w;
  const uint2 st = state[pair];
  const uint32_t T = st.x, r = st.y;
  // counts of the layer's chunks in front of this one
  if (threadIdx.x < 2) sh_base[threadIdx.x] = 0;
  __syncthreads();
  {
    const uint2* cc = chunk_cnt + static_cast<uint64_t>(w) * n_chunks;
    uint32_t g = 0, q = 0;
    for (uint32_t j = c.first_chunk_of_layer + threadIdx.x; j < blockIdx.x; j += THREADS) {
      const uint2 v = cc[j];
      if (chunk_sfx == nullptr) {  // (#keys > T, #keys == T) of the chunk, counted by a kernel of its own
        g += v.x;
        q += v.y;
      } else {  // left by the last histogram pass: keys above the prefix, suffix sums of the low digit
        constexpr uint32_t LOW_BINS = pass_bins(N_PASSES - 1);
        const uint32_t d = T & (LOW_BINS - 1);
        const uint32_t* sfx = chunk_sfx + (static_cast<uint64_t>(w) * n_chunks + j) * LOW_BINS;
        const uint32_t s_d = sfx[d], s_d1 = (d + 1 < LOW_BINS) ? sfx[d + 1] : 0u;
        g += v.x + s_d1;
        q += s_d - s_d1;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      g += __shfl_xor_sync(0xffffffffu, g, d);
      q += __shfl_xor_sync(0xffffffffu, q, d);
    }
    if ((threadIdx.x & 31) == 0 && (g | q)) {
      atomicAdd(&sh_base[0], g);
      atomicAdd(&sh_base[1], q);
    }
  }
  __syncthreads();
  uint32_t run_gt = sh_base[0], run_eq = sh_base[1];
  uint32_t* out_i = sel_idx + static_cast<uint64_t>(w) * K + L.koff;
  float* out_v = sel_val + static_cast<uint64_t>(w) * K + L.koff;

  const bool is_leader = w == leader;
  if (pair_is_cand(info[pair], L.k)) {
    // warp order is index order: count per warp, prefix over the warps, then every warp writes its
    // tiles front to back, ranking the entries of a slot with one warp scan per 128 entries
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t my_gt = 0, my_eq = 0;
    for_each_candidate(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      my_gt += key > T ? 1u : 0u;
      my_eq += key == T ? 1u : 0u;
    });
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      my_gt += __shfl_xor_sync(0xffffffffu, my_gt, d);
      my_eq += __shfl_xor_sync(0xffffffffu, my_eq, d);
    }
    __shared__ uint32_t sh_wg[WARPS], sh_we[WARPS];
    if (lane == 0) {
      sh_wg[warp] = my_gt;
      sh_we[warp] = my_eq;
    }
    __syncthreads();
    uint32_t g_before = run_gt, q_before = run_eq;
    for (uint32_t q = 0; q < warp; ++q) {
      g_before += sh_wg[q];
      q_before += sh_we[q];
    }
    if ((my_gt | my_eq) == 0) return;  // nothing of this warp's tiles is selected
    const uint32_t t_begin = warp * TILES_PER_WARP;
    const uint32_t t_end = min(c.n_tiles, t_begin + TILES_PER_WARP);
    // ranks the entries [j0, j0 + 128) of one slot with a warp scan and writes the selected ones
    auto emit = [&](uint32_t tile, uint64_t tw, uint32_t cnt, uint32_t tile_base, uint32_t j0, uint4 k) {
      const uint32_t j = j0 + lane * 4;
      const uint32_t kk[4] = {k.x, k.y, k.z, k.w};
      uint32_t fg = 0, fe = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {  // padding keys are 0 and T is not: no range test needed
        fg |= kk[u] > T ? (1u << u) : 0u;
        fe |= kk[u] == T ? (1u << u) : 0u;
      }
      if (!__any_sync(0xffffffffu, (fg | fe) != 0u)) return;
      // most entries of a slot are selected: fetch the group's values and indices as vectors now, so
      // that they arrive while the ranks are computed
      float4 v4 = make_float4(0.f, 0.f, 0.f, 0.f);
      uint2 i2 = make_uint2(0u, 0u);
      if (fg | fe) {
        v4 = reinterpret_cast<const float4*>(cand_val + tw * CAND_CAP)[j >> 2];
        i2 = reinterpret_cast<const uint2*>(cand_idx + tw * CAND_CAP)[j >> 2];
      }
      const uint32_t packed = static_cast<uint32_t>(__popc(fg)) | (static_cast<uint32_t>(__popc(fe)) << 16);
      const uint32_t incl = warp_incl_scan(packed);
      const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
      uint32_t gb = g_before + ((incl - packed) & 0xffffu), qb = q_before + ((incl - packed) >> 16);
      if (fg | fe) {
        const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
        const uint32_t ii[4] = {i2.x & 0xffffu, i2.x >> 16, i2.y & 0xffffu, i2.y >> 16};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool isg = (fg >> u) & 1u, ise = (fe >> u) & 1u;
          if (isg || (ise && qb < r)) {
            const uint32_t pos = gb + (qb < r ? qb : r);
            if (pos < L.k) {
              out_i[pos] = tile_base + ii[u];
              out_v[pos] = vv[u];
              if (is_leader) sel_slot[L.koff + pos] = tile * CAND_CAP + j + u;
            } else {
              atomicMin(status, STATUS_INTERNAL);
            }
          }
          gb += isg ? 1u : 0u;
          qb += ise ? 1u : 0u;
        }
      }
      g_before += tot & 0xffffu;
      q_before += tot >> 16;
    };
    for (uint32_t tb = t_begin; tb < t_end; tb += 4) {  // four tiles per batch, all their loads first
      uint32_t cnt[4], tbase[4];
      uint4 k4[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const bool in = tb + q < t_end;
        const uint32_t tile = c.first_tile + tb + q;
        cnt[q] = in ? min(cand_cnt[static_cast<uint64_t>(tile) * W + w], CAND_CAP) : 0u;
        tbase[q] = in ? (tiles[tile].a & ~(TILE - 1u)) : 0u;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t tw = static_cast<uint64_t>(c.first_tile + tb + q) * W + w;
        k4[q] = (lane * 4 < cnt[q]) ? reinterpret_cast<const uint4*>(cand_key + tw * CAND_CAP)[lane]
                                    : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (cnt[q] == 0) continue;
        const uint32_t tile = c.first_tile + tb + q;
        const uint64_t tw = static_cast<uint64_t>(tile) * W + w;
        emit(tile, tw, cnt[q], tbase[q], 0, k4[q]);
        for (uint32_t j0 = 128; j0 < cnt[q]; j0 += 128) {
          const uint32_t j = j0 + lane * 4;
          const uint4 k = (j < cnt[q]) ? reinterpret_cast<const uint4*>(cand_key + tw * CAND_CAP)[j >> 2]
                                       : make_uint4(0u, 0u, 0u, 0u);
          emit(tile, tw, cnt[q], tbase[q], j0, k);
        }
      }
    }
    return;
  }

  const uint64_t lo = c.a, hi = lo + c.len;
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  const float* a = acc + static_cast<uint64_t>(w) * N;
  for (uint32_t it = 0; it < n_iter; ++it) {
    const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
    float av[4], wv[4];
    load4<VEC>(a, e0, lo, hi, av);
    load4<VEC>(weights, e0, lo, hi, wv);
    uint32_t fg = 0, fe = 0;  // per-element flags
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint64_t e = e0 + q;
      const bool in = e >= lo && e < hi;
      const uint32_t key = imp_key(av[q], wv[q], eps);
      fg |= (in && key > T) ? (1u << q) : 0u;
      fe |= (in && key == T) ? (1u << q) : 0u;
    }
    uint32_t total;
    const uint32_t packed = static_cast<uint32_t>(__popc(fg)) | (static_cast<uint32_t>(__popc(fe)) << 16);
    const uint32_t ex = block_excl_scan(packed, sh_warp, total);
    uint32_t g_before = run_gt + (ex & 0xffffu), q_before = run_eq + (ex >> 16);
    if (fg | fe) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const bool isg = (fg >> q) & 1u, ise = (fe >> q) & 1u;
        if (isg || (ise && q_before < r)) {
          const uint32_t pos = g_before + (q_before < r ? q_before : r);
          if (pos < L.k) {
            out_i[pos] = static_cast<uint32_t>(e0 + q);
            out_v[pos] = av[q];
            if (is_leader) sel_slot[L.koff + pos] = REF_LAZY;
          } else {
            atomicMin(status, STATUS_INTERNAL);
          }
        }
        g_before += isg ? 1u : 0u;
        q_before += ise ? 1u : 0u;
      }
    }
    run_gt += total & 0xffffu;
    run_eq += total >> 16;
  }
}

// ---------------------------------------------------------------------------------------
// one-CTA path: steps (a)-(d) of a whole (worker, layer) pair with n <= SMALL_MAX, keys in
// shared memory.  grid = (small layers, W); dynamic shared memory = 4 * max n bytes.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS)
    k_small(const float* __restrict__ grads, const float* __restrict__ weights, float* __restrict__ acc,
            float* __restrict__ update, const LayerDesc* __restrict__ layers, const uint32_t* __restrict__ small_ids,
            uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val, uint32_t* __restrict__ sel_slot,
            int* __restrict__ status, float eps, uint64_t N, uint64_t K, int leader, float momentum) {
  extern __shared__ uint32_t keys[];
  __shared__ uint32_t hist[NBINS];
  __shared__ uint32_t sh_scan[THREADS];
  __shared__ uint32_t sh_warp[WARPS];
  __shared__ uint32_t res[4];
  const LayerDesc L = layers[small_ids[blockIdx.x]];
  const int w = blockIdx.y;
  const int tid = threadIdx.x;
  const uint32_t n = L.n;
  float* a = acc + static_cast<uint64_t>(w) * N + L.off;
  const float* g = grads + static_cast<uint64_t>(w) * N + L.off;
  const float* wt = weights + L.off;
  for (uint32_t i = tid; i < n; i += THREADS) {
    const float v = accumulate(a[i], __ldcs(g + i), momentum);
    a[i] = v;
    keys[i] = imp_key(v, wt[i], eps);
    if (w == 0) update[L.off + i] = 0.0f;
  }
  __syncthreads();
  uint32_t T, r;
  if (!smem_radix_select(keys, n, L.k, hist, sh_scan, res, T, r)) {
    if (tid == 0) atomicMin(status, STATUS_INTERNAL);
    return;
  }
  uint32_t* out_i = sel_idx + static_cast<uint64_t>(w) * K + L.koff;
  float* out_v = sel_val + static_cast<uint64_t>(w) * K + L.koff;
  uint32_t run_gt = 0, run_eq = 0;
  for (uint32_t i0 = 0; i0 < n; i0 += THREADS) {
    const uint32_t i = i0 + tid;
    const uint32_t key = i < n ? keys[i] : 0u;
    const bool isg = i < n && key > T, ise = i < n && key == T;
    uint32_t total;
    const uint32_t ex = block_excl_scan((isg ? 1u : 0u) | (ise ? 1u << 16 : 0u), sh_warp, total);
    const uint32_t g_before = run_gt + (ex & 0xffffu), q_before = run_eq + (ex >> 16);
    if (isg || (ise && q_before < r)) {
      const uint32_t pos = g_before + (q_before < r ? q_before : r);
      if (pos < L.k) {
        out_i[pos] = L.off + i;
        out_v[pos] = a[i];
        if (w == leader) sel_slot[L.koff + pos] = REF_NONE;
      } else {
        atomicMin(status, STATUS_INTERNAL);
      }
    }
    run_gt += total & 0xffffu;
    run_eq += total >> 16;
  }
}

// ---------------------------------------------------------------------------------------
// steps (e)-(g): gather every worker's residual at the leader's indices, sum in ascending
// worker order, scatter into the (already zeroed) dense update, zero what was sent.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS)
    k_gather_sum_scatter(const uint32_t* __restrict__ leader_idx, float* __restrict__ acc, float* __restrict__ update,
                         uint64_t N, uint64_t K, int W) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= K) return;
  const uint64_t i = leader_idx[j];
  float* p = acc + i;
  float s = 0.0f;
  for (int w0 = 0; w0 < W; w0 += 8) {  // loads of a group are independent; the sum keeps worker order
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = (w0 + u < W) ? p[static_cast<uint64_t>(w0 + u) * N] : 0.0f;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (w0 + u < W) s = (w0 + u == 0) ? v[u] : __fadd_rn(s, v[u]);
    }
  }
  for (int w = 0; w < W; ++w) p[static_cast<uint64_t>(w) * N] = 0.0f;
  update[i] = __fadd_rn(0.0f, s);
}

// Steps (e)-(g) with several chosen nodes (Algorithm 1: Mask = OR Mask_ri): the index set is the union
// of the chosen nodes' lists.  One thread per list entry of every chosen node; the first thread to mark
// an element in the (all-zero) bit mask owns it - gathers the W residuals, sums them in ascending
// worker order, scatters the sum and zeroes the residuals - and every later entry with the same element
// returns at once, so nothing is read after it was zeroed.  The marks stay set (the element is +0 now
// whether or not the next streaming pass treats it so).
__global__ void __launch_bounds__(THREADS)
    k_union_sum_scatter(const uint32_t* __restrict__ sel_idx, float* __restrict__ acc, float* __restrict__ update,
                        uint32_t* __restrict__ seen, uint64_t N, uint64_t K, int W, LeaderSet ls) {
  const uint64_t q = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (q >= static_cast<uint64_t>(ls.n) * K) return;
  const int j = static_cast<int>(q / K);
  int r = ls.r[0];
#pragma unroll
  for (int u = 1; u < MAX_LEADERS; ++u)
    if (u == j) r = ls.r[u];
  const uint64_t i = sel_idx[static_cast<uint64_t>(r) * K + q % K];
  const uint32_t bit = zmask_bit(i);
  if (atomicOr(&seen[zmask_word(i)], bit) & bit) return;
  float* p = acc + i;
  float s = 0.0f;
  for (int w0 = 0; w0 < W; w0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = (w0 + u < W) ? p[static_cast<uint64_t>(w0 + u) * N] : 0.0f;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (w0 + u < W) s = (w0 + u == 0) ? v[u] : __fadd_rn(s, v[u]);
    }
  }
  for (int w = 0; w < W; ++w) p[static_cast<uint64_t>(w) * N] = 0.0f;
  update[i] = __fadd_rn(0.0f, s);
}

// Workers spread over several contexts (one per GPU): step (e) for this context's workers at an index
// set that came from elsewhere, vals[w][j] = acc[w][idx[j]]; grid-stride over (worker, entry).
__global__ void __launch_bounds__(THREADS)
    k_shard_gather(const uint32_t* __restrict__ idx, const float* __restrict__ acc, float* __restrict__ vals, uint64_t N,
                   uint64_t n, int W) {
  const uint64_t total = n * static_cast<uint64_t>(W);
  for (uint64_t q = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x; q < total;
       q += static_cast<uint64_t>(gridDim.x) * THREADS) {
    const uint64_t w = q / n, j = q % n;
    vals[q] = acc[w * N + idx[j]];
  }
}

// ... and steps (f), (g): the values of ALL workers of the job at the index set, in global worker order
// (vals_all[w][j], w < W_total), are summed in that order into the (already zeroed) update, and this
// context's own residuals are zeroed there.  One thread per entry.
__global__ void __launch_bounds__(THREADS)
    k_shard_apply(const uint32_t* __restrict__ idx, const float* __restrict__ vals_all, float* __restrict__ acc,
                  float* __restrict__ update, uint64_t N, uint64_t n, int W_total, int W_local) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= n) return;
  const uint64_t i = idx[j];
  float s = vals_all[j];
  for (int w = 1; w < W_total; ++w) s = __fadd_rn(s, vals_all[static_cast<uint64_t>(w) * n + j]);
  update[i] = __fadd_rn(0.0f, s);
  for (int w = 0; w < W_local; ++w) acc[static_cast<uint64_t>(w) * N + i] = 0.0f;
}

// A worker's select that is left running on a side stream past the end of the step may still need
// the weights if its pair has to fall back to the multi-pass path, and the caller is free to change
// them once the step's stream work is done.  So the weights of every layer in which a worker other
// than the leader failed its single-read check are copied here, on the step's own stream; that
// select then reads the copy.  grid = chunks; nearly always every CTA returns at once.
__global__ void __launch_bounds__(THREADS)
    k_save_weights(const float* __restrict__ weights, float* __restrict__ saved, const Chunk* __restrict__ chunks,
                   const LayerDesc* __restrict__ layers, const PairInfo* __restrict__ info, int W, int leader) {
  const Chunk c = chunks[blockIdx.x];
  const LayerDesc L = layers[c.layer];
  bool failed = false;
  for (int w = threadIdx.x; w < W; w += THREADS)
    failed = failed || (w != leader && !pair_is_cand(info[static_cast<uint32_t>(L.large_index) * W + w], L.k));
  if (!__syncthreads_or(failed)) return;
  for (uint32_t i = threadIdx.x; i < c.len; i += THREADS) saved[c.a + i] = weights[c.a + i];
}

// Steps (e)-(g) on the single-read path.  For a list entry of the leader that came from a candidate
// slot, every other worker's value at that slot position was written to the side buffer by the
// streaming pass (the leader's own value is the candidate value): read the W values, sum them in
// ascending worker order, scatter, and mark the element for zeroing by the next streaming pass.
// Entries from the one-CTA path carry REF_NONE: gathered from the residuals, which are zeroed here
// (no streaming pass visits them).  Entries from a pair that fell back to the multi-pass select
// carry REF_LAZY: gathered from the residuals and marked like the first kind, because another
// worker's multi-pass select may still be reading that layer's residuals on a side stream.
__global__ void __launch_bounds__(THREADS)
    k_sum_scatter(const uint32_t* __restrict__ leader_idx, const uint32_t* __restrict__ sel_slot,
                  const float* __restrict__ side_val, const float* __restrict__ cand_val, float* __restrict__ acc,
                  float* __restrict__ update, uint32_t* __restrict__ zmask, uint64_t N, uint64_t K, int W,
                  int leader) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= K) return;
  const uint64_t i = leader_idx[j];
  const uint32_t ref = sel_slot[j];
  float s = 0.0f;
  if (ref < REF_LAZY) {
    const uint64_t tile = ref / CAND_CAP, at = ref % CAND_CAP;
    const uint64_t q0 = tile * W * CAND_CAP + at;
    for (int w0 = 0; w0 < W; w0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int w = w0 + u;
        const uint64_t q = q0 + static_cast<uint64_t>(w) * CAND_CAP;
        v[u] = (w < W) ? (w == leader ? cand_val[q] : side_val[q]) : 0.0f;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (w0 + u < W) s = (w0 + u == 0) ? v[u] : __fadd_rn(s, v[u]);
      }
    }
    atomicOr(&zmask[zmask_word(i)], zmask_bit(i));  // the next streaming pass zeroes all W residuals
  } else {
    float* p = acc + i;
    for (int w0 = 0; w0 < W; w0 += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = (w0 + u < W) ? p[static_cast<uint64_t>(w0 + u) * N] : 0.0f;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (w0 + u < W) s = (w0 + u == 0) ? v[u] : __fadd_rn(s, v[u]);
      }
    }
    if (ref == REF_LAZY) {
      atomicOr(&zmask[zmask_word(i)], zmask_bit(i));
    } else {
      for (int w = 0; w < W; ++w) p[static_cast<uint64_t>(w) * N] = 0.0f;
    }
  }
  update[i] = __fadd_rn(0.0f, s);
}

// Applies a pending zero mask right away (accessors, reset, and the multi-pass path need the
// residuals themselves up to date).  One thread per mask word; the mask is cleared.
__global__ void __launch_bounds__(THREADS)
    k_flush_zmask(uint32_t* __restrict__ zmask, float* __restrict__ acc, uint64_t n_words, uint64_t N, int W) {
  const uint64_t wd = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (wd >= n_words) return;
  uint32_t bits = zmask[wd];
  if (bits == 0u) return;
  zmask[wd] = 0u;
  const uint64_t field0 = wd * 2;  // (segment, lane) index of the low half
  for (; bits; bits &= bits - 1) {
    const uint32_t b = __ffs(bits) - 1;
    const uint64_t field = field0 + (b >> 4);
    const uint64_t seg = field >> 5, lane = field & 31;
    const uint32_t fb = b & 15u;
    const uint64_t i = seg * 512 + (fb >> 2) * 128 + lane * 4 + (fb & 3u);
    if (i < N) {
      for (int w = 0; w < W; ++w) acc[static_cast<uint64_t>(w) * N + i] = 0.0f;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Absolute-threshold mode: Algorithm 1 as printed.  Only the chosen nodes form masks, per layer
// Mask = |G / w| > thr (strict; several nodes' masks are OR-ed), and the index set has whatever size
// results.  A step: step (a) for the chosen nodes (k_thr_accumulate_chosen), two looks at their
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
__device__ __forceinline__ bool thr_selected(float acc, float w, float eps, uint32_t T, uint64_t e,
                                             const RandomSelect& rs) {
  const uint32_t key = imp_key(acc, w, eps);
  // importance patterns are non-negative, so as signed integers they order like the values against any
  // threshold pattern: a negative threshold (layer-wise mode can produce one) is below every importance
  if (static_cast<int32_t>(key) > static_cast<int32_t>(T)) return true;
  if (!rs.on) return false;
  const float u = __fmul_rn(static_cast<float>(draw24(rs.seed, rs.step, e)), 5.9604644775390625e-08f);
  return u < __fdiv_rn(__uint_as_float(key), __uint_as_float(T));
}

template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_thr_count(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
                const uint32_t* __restrict__ thr_bits, uint32_t thr_stride, uint32_t* __restrict__ chunk_cnt, float eps,
                uint64_t N, LeaderSet ls, RandomSelect rs) {
  __shared__ uint32_t sh_cnt;
  const Chunk c = chunks[blockIdx.x];
  // thr_stride = 0: one threshold per layer for every chosen node; = number of layers: node j has its own row
  const uint32_t* T = thr_bits + c.layer;
  if (threadIdx.x == 0) sh_cnt = 0;
  __syncthreads();
  const uint64_t lo = c.a, hi = lo + c.len;
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  uint32_t cnt = 0;
  for (uint32_t it = 0; it < n_iter; ++it) {
    const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
    float wv[4];
    load4<VEC>(weights, e0, lo, hi, wv);
    uint32_t f = 0;  // Mask = OR of the chosen nodes' masks
    for (int j = 0; j < ls.n; ++j) {
      float av[4];
      load4<VEC>(acc + static_cast<uint64_t>(ls.r[j]) * N, e0, lo, hi, av);
#pragma unroll
      for (int q = 0; q < 4; ++q) f |= thr_selected(av[q], wv[q], eps, T[j * thr_stride], e0 + q, rs) ? (1u << q) : 0u;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint64_t e = e0 + q;
      cnt += (e >= lo && e < hi && ((f >> q) & 1u)) ? 1u : 0u;
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

template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_thr_write(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
                const uint32_t* __restrict__ thr_bits, uint32_t thr_stride, const uint32_t* __restrict__ chunk_off,
                uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val, uint32_t capacity,
                int* __restrict__ status, uint32_t* __restrict__ set_bits, float eps, uint64_t N, LeaderSet ls,
                RandomSelect rs) {
  __shared__ uint32_t sh_warp[WARPS];
  const Chunk c = chunks[blockIdx.x];
  const uint32_t* T = thr_bits + c.layer;
  uint32_t run = chunk_off[blockIdx.x];
  const uint64_t lo = c.a, hi = lo + c.len;
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  for (uint32_t it = 0; it < n_iter; ++it) {
    const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + threadIdx.x) * 4;
    float av[4], wv[4];  // av: r_1's values, the ones listed
    load4<VEC>(acc + static_cast<uint64_t>(ls.r[0]) * N, e0, lo, hi, av);
    load4<VEC>(weights, e0, lo, hi, wv);
    uint32_t f = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) f |= thr_selected(av[q], wv[q], eps, T[0], e0 + q, rs) ? (1u << q) : 0u;
    for (int j = 1; j < ls.n; ++j) {
      float bv[4];
      load4<VEC>(acc + static_cast<uint64_t>(ls.r[j]) * N, e0, lo, hi, bv);
#pragma unroll
      for (int q = 0; q < 4; ++q) f |= thr_selected(bv[q], wv[q], eps, T[j * thr_stride], e0 + q, rs) ? (1u << q) : 0u;
    }
    {
      uint32_t inside = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) inside |= (e0 + q >= lo && e0 + q < hi) ? (1u << q) : 0u;
      f &= inside;
    }
    // the index set as a bit per element (zeroed before the step) for the fused pass over all workers;
    // a slot's four bits never straddle a word because slots start at multiples of four
    if (f) atomicOr(&set_bits[e0 >> 5], f << (e0 & 31u));
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
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_thr_stats(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
                unsigned long long* __restrict__ bins, float eps, uint64_t N, uint32_t n_layers, LeaderSet ls) {
  __shared__ unsigned long long sh[3 * LW_BINS];
  __shared__ unsigned long long sh_fast[8];  // digits: [0..2] first moment, [3..7] second
  __shared__ uint32_t sh_exp[2];             // sum and count of the exponents sampled for the window
  const Chunk c = chunks[blockIdx.x];
  const int j = blockIdx.y;
  int r = ls.r[0];
#pragma unroll
  for (int q = 1; q < MAX_LEADERS; ++q)
    if (q == j) r = ls.r[q];
  for (int b = threadIdx.x; b < 3 * LW_BINS; b += THREADS) sh[b] = 0ull;
  if (threadIdx.x < 8) sh_fast[threadIdx.x] = 0ull;
  if (threadIdx.x < 2) sh_exp[threadIdx.x] = 0u;
  __syncthreads();
  const float* a = acc + static_cast<uint64_t>(r) * N;
  const uint64_t lo = c.a, hi = lo + c.len;
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  const int lane = threadIdx.x & 31;
  // widest shift that keeps m << d inside 63 bits summed over this thread's elements (and m^2 << 2d inside 127)
  const int d_max = min(30, 39 - (32 - __clz(n_iter * 4)));
  int base = 1;
  {  // window: average exponent of the first element of every thread, minus 14
    const uint64_t e = s0 + static_cast<uint64_t>(threadIdx.x) * 4;
    uint32_t f = 0, cnt = 0;
    for (int q = 0; q < 4 && cnt == 0; ++q) {
      if (e + q >= lo && e + q < hi) {
        const uint32_t key = imp_key(a[e + q], weights[e + q], eps);
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
  // the threads' window sums, digit by digit (each digit sum stays far below 2^64)
  if (s1) {
    atomicAdd(&sh_fast[0], s1 & 0xffffffffull);
    atomicAdd(&sh_fast[1], s1 >> 32);
  }
  if (s2) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const unsigned long long dg = static_cast<unsigned long long>(s2 >> (32 * k)) & 0xffffffffull;
      if (dg) atomicAdd(&sh_fast[3 + k], dg);
    }
  }
  __syncthreads();
  unsigned long long* g = bins + (static_cast<uint64_t>(j) * n_layers + c.layer) * (3 * LW_BINS);
  for (int b = threadIdx.x; b < 3 * LW_BINS; b += THREADS) {
    const unsigned long long v = sh[b];
    if (v) atomicAdd(&g[b], v);
  }
  if (threadIdx.x < 2 && sh_fast[threadIdx.x]) atomicAdd(&g[base + 32 * threadIdx.x], sh_fast[threadIdx.x]);
  if (threadIdx.x >= 3 && threadIdx.x < 7 && sh_fast[threadIdx.x])
    atomicAdd(&g[2 * LW_BINS + base + 16 * (threadIdx.x - 3)], sh_fast[threadIdx.x]);
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

// Threshold mode, first pass: step (a) for the chosen nodes only (their masks are needed before anybody
// else's residual is touched).  grid = tiles.
template <bool VEC>
__global__ void __launch_bounds__(THREADS)
    k_thr_accumulate_chosen(const float* __restrict__ grads, float* __restrict__ acc, const Tile* __restrict__ tiles,
                            uint64_t N, float momentum, LeaderSet ls) {
  const Tile t = tiles[blockIdx.x];
  const uint64_t lo = t.a, hi = lo + t.len;
  const uint64_t base = lo & ~static_cast<uint64_t>(TILE - 1);
  constexpr int SPT = TILE / 4 / THREADS;
  for (int j = 0; j < ls.n; ++j) {
    const float* g = grads + static_cast<uint64_t>(ls.r[j]) * N;
    float* a = acc + static_cast<uint64_t>(ls.r[j]) * N;
    float gv[SPT][4], av[SPT][4];
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
      const uint64_t e0 = base + static_cast<uint64_t>(s * THREADS + threadIdx.x) * 4;
      load4_stream<VEC>(g, e0, lo, hi, gv[s]);
      load4_stream<VEC>(a, e0, lo, hi, av[s]);
    }
#pragma unroll
    for (int s = 0; s < SPT; ++s) {
      const uint64_t e0 = base + static_cast<uint64_t>(s * THREADS + threadIdx.x) * 4;
#pragma unroll
      for (int c = 0; c < 4; ++c) av[s][c] = accumulate(av[s][c], gv[s][c], momentum);
      store4<VEC>(a, e0, lo, hi, av[s]);
    }
  }
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

// byte mask of the index set (Algorithm 1's encode_uint8(Mask)); dst is zeroed by the caller
__global__ void __launch_bounds__(THREADS) k_mask_scatter(const uint32_t* __restrict__ leader_idx, uint8_t* __restrict__ dst, uint64_t K) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j < K) dst[leader_idx[j]] = 1;
}

}  // namespace iwp

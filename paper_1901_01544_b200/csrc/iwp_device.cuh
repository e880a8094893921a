// Device-side helpers shared by all kernels of the pruning step: constants, the per-pair record of the
// single-read path, worker subsets, the IEEE importance arithmetic, 128-bit load/store helpers, warp and
// block scans, the shared-memory radix select and the warp-aggregated histogram add.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_plan.hpp"

namespace iwp {

constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int STATUS_INTERNAL = -4;
constexpr int STATUS_CAPACITY = -6;

// Debug build (-DIWP_DEBUG_CHECKS, `python -m paper_1901_01544_b200.build --debug`): every computed index is
// range-checked and the histogram counts are checked for conservation; a failed check sets the status word
// (nothing traps).  In the release build the checks compile to nothing.
#ifdef IWP_DEBUG_CHECKS
#define IWP_DBG_CHECK(status, cond)                          \
  do {                                                       \
    if (!(cond)) atomicMin((status), STATUS_INTERNAL);       \
  } while (0)
constexpr bool DEBUG_CHECKS = true;
#else
#define IWP_DBG_CHECK(status, cond) \
  do {                              \
  } while (0)
constexpr bool DEBUG_CHECKS = false;
#endif

// radix-select digit plan over the 32-bit importance pattern (bit 31 is always 0)
__host__ __device__ constexpr int pass_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__host__ __device__ constexpr int pass_bins(int pass) { return pass == 2 ? 1024 : 2048; }
constexpr int N_PASSES = 3;

// Per (tiled layer, worker) pair: the threshold guess of the single-read path and what the
// fused accumulate pass found with it.
struct PairInfo {
  uint32_t guess;  // candidates include every element with importance pattern >= guess; GUESS_NONE = none
  uint32_t total;  // number of elements of the layer that reach the guess
  uint32_t flags;  // bit 0: some (tile, worker) slot overflowed
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

// Exclusive prefix sum over the block (NW warps) in thread order; `total` = block sum.
// sh_warp: NW words of shared memory.  Contains two __syncthreads().
template <int NW = WARPS>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t x, uint32_t* sh_warp, uint32_t& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const uint32_t incl = warp_incl_scan(x);
  if (lane == 31) sh_warp[wid] = incl;
  __syncthreads();
  uint32_t woff = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < NW; ++i) {
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
// res[0] = d, res[1] = krem - count(digit > d), res[2] = 1 if found.  sh_scan: NT / 32 words.
// Suffix sums over the threads' bin groups: by shuffles inside a warp, then over the warps' totals
// (two block barriers in all).
template <int NT = THREADS>
__device__ __forceinline__ void find_digit(const uint32_t* hist, int nb, uint32_t krem, uint32_t* sh_scan,
                                           uint32_t* res) {
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  constexpr int NW = NT / 32;
  const int per = nb / NT;
  uint32_t local = 0;
  for (int b = 0; b < per; ++b) local += hist[tid * per + b];
  uint32_t incl = local;  // inclusive suffix sum over the lanes of the warp
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t y = __shfl_down_sync(0xffffffffu, incl, d);
    if (lane + d < 32) incl += y;
  }
  if (lane == 0) sh_scan[wid] = incl;
  if (tid == 0) res[2] = 0;
  __syncthreads();
  for (int i = wid + 1; i < NW; ++i) incl += sh_scan[i];  // the warps above this one
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

// Pre-test multiplier of the single-read path: with gm = guess * (1 - 2^-20) every element whose correctly
// rounded quotient |acc| / den reaches the guess passes |acc| >= gm * den (the two roundings of gm * den and the
// one of the quotient are each below 2^-23 relative).  The argument needs normal products, so the pre-test is
// disabled (gm = 0: everything passes) for tiny guesses or eps; +inf = no guess, nothing passes.
__device__ __forceinline__ float pretest_multiplier(uint32_t guess, float eps) {
  if (guess == GUESS_NONE) return __int_as_float(0x7f800000);  // +inf: nothing passes
  const float gf = __uint_as_float(guess);
  const float tiny = 8.673617379884035e-19f;  // 2^-60
  if (!(gf >= tiny) || !(eps >= tiny)) return 0.0f;
  return __fmul_rd(gf, 1.0f - 9.5367431640625e-07f);
}

// Warp-aggregated increment of a shared-memory histogram: lanes that hit the same bin
// elect one lane that adds the whole group's count.  Must be called by all 32 lanes.
__device__ __forceinline__ void hist_add_aggregated(uint32_t* hist, bool valid, uint32_t bin) {
  const uint32_t tag = valid ? bin : 0xffffffffu;
  const uint32_t peers = __match_any_sync(0xffffffffu, tag);
  const int lane = threadIdx.x & 31;
  if (valid && (__ffs(peers) - 1) == lane) atomicAdd(&hist[bin], static_cast<uint32_t>(__popc(peers)));
}

}  // namespace iwp

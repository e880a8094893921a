// Steps (c)+(d) of the pruning step: exact radix select over the fp32 importance pattern (histogram passes,
// digit decisions), ordered compaction into the (index, value) lists, and the one-CTA path of small layers.
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_device.cuh"
#include "iwp_stream.cuh"

namespace iwp {

// CTA size of the select kernels (histogram passes, digit decisions, compaction).  Four warps of at most 64
// registers: such a CTA fits into the registers three CTAs of the streaming pass leave free on an SM (7 warps x
// 80 registers each in the other workers' launch: 53 760 of 65 536), so a select that runs beside the streaming
// pass takes no CTA slot away from it.
constexpr int SEL_THREADS = 128;
constexpr int SEL_WARPS = SEL_THREADS / 32;

// The candidates of (chunk, worker): warp q takes the q-th eighth of the chunk's tiles (consecutive,
// so that warp order is index order), four tiles at a time; each lane reads entries 4 lane .. 4 lane + 3
// of a slot with one 128-bit load (a slot rarely holds more than 128 entries; a tail loop covers the
// rest) and all loads of a batch are issued before any is used.  `f(key)` sees every stored candidate,
// and in addition some keys 0 (padding, slots shorter than 128 entries), which `f` must ignore - every
// use below does so by construction, because a candidate's key and first digit are never 0.
template <int NW>
__device__ __forceinline__ uint32_t tiles_per_warp(const Chunk& c) { return (c.n_tiles + NW - 1) / NW; }

template <int NW = SEL_WARPS, typename F>
__device__ __forceinline__ void for_each_candidate(const Chunk& c, int w, int W, const uint32_t* __restrict__ cand_cnt,
                                                   const uint32_t* __restrict__ cand_key, F&& f) {
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t t_begin = min(c.n_tiles, warp * tiles_per_warp<NW>(c));
  const uint32_t t_end = min(c.n_tiles, t_begin + tiles_per_warp<NW>(c));
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
template <bool VEC, int NW>
__global__ void __launch_bounds__(NW * 32, 512 / (NW * 32) * 2)
    k_hist(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
           const LayerDesc* __restrict__ layers, const PairInfo* __restrict__ info,
           const uint32_t* __restrict__ cand_key, const uint32_t* __restrict__ cand_cnt,
           const uint2* __restrict__ state,
           uint32_t* __restrict__ hist, uint32_t* __restrict__ chunk_sfx, uint2* __restrict__ chunk_cnt,
           uint32_t* __restrict__ reach_seen, float eps, uint64_t N, int W, int pass, uint32_t n_chunks, WorkerSel ws,
           const uint32_t* __restrict__ chunk_ids) {
  __shared__ uint32_t sh[NBINS];
  __shared__ uint32_t sh_warp[NW];
  __shared__ uint32_t sh_above;
  // the chunks this launch covers: all of them, or (chunk_ids) those of the layers the chain selects
  const uint32_t ci = chunk_ids != nullptr ? chunk_ids[blockIdx.x] : blockIdx.x;
  const Chunk c = chunks[ci];
  const int w = sel_worker(ws, static_cast<int>(blockIdx.y));
  const LayerDesc L = layers[c.layer];
  const uint32_t pair = static_cast<uint32_t>(L.large_index) * W + w;
  const int shift = pass_shift(pass), nb = pass_bins(pass);
  const int prev_shift = pass == 0 ? 31 : pass_shift(pass - 1);
  const uint2 st_in = pass == 0 ? make_uint2(0u, L.k) : state[pair];
  const uint32_t want = pass == 0 ? 0u : (st_in.x >> prev_shift);
  const bool last_pass = pass == N_PASSES - 1;
  for (int b = threadIdx.x; b < nb; b += (NW * 32)) sh[b] = 0;
  if (threadIdx.x == 0) sh_above = 0;
  __syncthreads();
  uint32_t above = 0;  // keys whose higher digits already exceed the prefix (needed in the last pass only)
  const PairInfo pi = info[pair];
  if (pair_is_cand(pi, L.k) && pass == 0) {
    // Every candidate is at or just above the guess, so almost all of them fall into the guess's own
    // first-digit bin or the next two: count those in registers (one shared-memory atomic per lane
    // would serialise on three addresses) and leave only the rest to atomics.
    const uint32_t g0 = pi.guess >> shift;
    // Conservation check: the stored entries that reach the guess are counted again here and must add up
    // to the number the streaming pass counted when it stored them (k_find_digit compares).
    uint32_t c0 = 0, c1 = 0, c2 = 0, ge = 0;
    for_each_candidate<NW>(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      const uint32_t d = (key >> shift) - g0;
      c0 += d == 0u ? 1u : 0u;
      c1 += d == 1u ? 1u : 0u;
      c2 += d == 2u ? 1u : 0u;
      ge += key >= pi.guess ? 1u : 0u;
      if (d > 2u && key != 0u) atomicAdd(&sh[(key >> shift) & (nb - 1)], 1u);
    });
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      c0 += __shfl_xor_sync(0xffffffffu, c0, d);
      c1 += __shfl_xor_sync(0xffffffffu, c1, d);
      c2 += __shfl_xor_sync(0xffffffffu, c2, d);
      ge += __shfl_xor_sync(0xffffffffu, ge, d);
    }
    if ((threadIdx.x & 31) == 0) {
      if (c0) atomicAdd(&sh[g0 & (nb - 1)], c0);
      if (c1) atomicAdd(&sh[(g0 + 1) & (nb - 1)], c1);
      if (c2) atomicAdd(&sh[(g0 + 2) & (nb - 1)], c2);
      if (ge && reach_seen != nullptr) atomicAdd(&reach_seen[pair], ge);
    }
  } else if (pair_is_cand(pi, L.k)) {
    for_each_candidate<NW>(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      const uint32_t hi_part = key >> prev_shift;
      if (hi_part == want) atomicAdd(&sh[(key >> shift) & (nb - 1)], 1u);
      above += hi_part > want ? 1u : 0u;
    });
  } else {
    const uint64_t lo = c.a, hi = lo + c.len;
    const uint64_t s0 = lo & ~3ull;
    const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + (NW * 32) * 4 - 1) / ((NW * 32) * 4));
    const float* a = acc + static_cast<uint64_t>(w) * N;
    for (uint32_t it = 0; it < n_iter; ++it) {
      const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * (NW * 32) + threadIdx.x) * 4;
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
  for (int b = threadIdx.x; b < nb; b += (NW * 32)) {
    const uint32_t v = sh[b];
    if (v) atomicAdd(&gh[b], v);
  }
  if (last_pass && chunk_sfx != nullptr) {  // suffix sums S[b] = sum of this chunk's bins >= b, and the count above the prefix
    constexpr int BPT = pass_bins(N_PASSES - 1) / (NW * 32);  // bins per thread in the last pass
    static_assert(BPT >= 2 && BPT * (NW * 32) == pass_bins(N_PASSES - 1), "a whole number of bins per thread");
    uint32_t h[BPT], mine = 0;
#pragma unroll
    for (int q = 0; q < BPT; ++q) {
      h[q] = sh[threadIdx.x * BPT + q];
      mine += h[q];
    }
    uint32_t total;
    const uint32_t before = block_excl_scan<NW>(mine, sh_warp, total);
    uint32_t run = total - before;  // sum of the bins >= this thread's first one
    uint32_t* dst = chunk_sfx + (static_cast<uint64_t>(w) * n_chunks + ci) * pass_bins(N_PASSES - 1);
    if constexpr (BPT % 4 == 0) {
#pragma unroll
      for (int q = 0; q < BPT; q += 4) {
        const uint4 sfx = make_uint4(run, run - h[q], run - h[q] - h[q + 1], run - h[q] - h[q + 1] - h[q + 2]);
        reinterpret_cast<uint4*>(dst)[(threadIdx.x * BPT + q) >> 2] = sfx;
        run -= h[q] + h[q + 1] + h[q + 2] + h[q + 3];
      }
    } else {
#pragma unroll
      for (int q = 0; q < BPT; q += 2) {
        reinterpret_cast<uint2*>(dst)[(threadIdx.x * BPT + q) >> 1] = make_uint2(run, run - h[q]);
        run -= h[q] + h[q + 1];
      }
    }
    if (threadIdx.x == 0) chunk_cnt[static_cast<uint64_t>(w) * n_chunks + ci] = make_uint2(sh_above, 0u);
  }
}

// Digit decision for (worker, layer) pairs of the tiled path; grid = (tiled layers, covered workers).
// Reads the pair's histogram, clears it for the next pass, extends the key prefix.
// After the last pass state = (threshold key T, number r of T-valued elements to keep).
template <int NW>
__global__ void __launch_bounds__(NW * 32, 512 / (NW * 32) * 2)
    k_find_digit(uint2* __restrict__ state, uint32_t* __restrict__ hist, const LayerDesc* __restrict__ layers,
                 const uint32_t* __restrict__ large_ids, const PairInfo* __restrict__ info,
                 uint32_t* __restrict__ reach_seen, int* __restrict__ status, int W, int pass, WorkerSel ws,
                 const uint32_t* __restrict__ large_sel) {
  __shared__ uint32_t sh[NBINS];
  __shared__ uint32_t sh_scan[(NW * 32)];
  __shared__ uint32_t res[4];
  // the tiled layers this launch covers: all of them, or (large_sel) those the chain selects
  const uint32_t li = large_sel != nullptr ? large_sel[blockIdx.x] : blockIdx.x;
  const uint32_t pair = li * static_cast<uint32_t>(W) + static_cast<uint32_t>(sel_worker(ws, static_cast<int>(blockIdx.y)));
  const int nb = pass_bins(pass), shift = pass_shift(pass);
  uint32_t* gh = hist + static_cast<uint64_t>(pair) * NBINS;
  for (int b = threadIdx.x; b < nb; b += (NW * 32)) {
    sh[b] = gh[b];
    gh[b] = 0;
  }
  __syncthreads();
  uint32_t prefix, krem;
  if (pass == 0) {
    prefix = 0;
    krem = layers[large_ids[pair / W]].k;
    if (DEBUG_CHECKS && info != nullptr && !pair_is_cand(info[pair], krem)) {
      // multi-pass path: the first histogram pass counted every element of the layer exactly once
      uint32_t part = 0;
      for (int b = threadIdx.x; b < nb; b += (NW * 32)) part += sh[b];
      uint32_t total;
      block_excl_scan<NW>(part, sh_scan, total);
      if (threadIdx.x == 0) IWP_DBG_CHECK(status, total == layers[large_ids[pair / W]].n);
    }
    if (threadIdx.x == 0 && reach_seen != nullptr) {
      // a pair that selects from its candidate slots: what the first histogram pass found in the slots must be
      // what the streaming pass put there (a lost, overwritten or stale entry shows up as a different count)
      const PairInfo pi = info[pair];
      const uint32_t seen = reach_seen[pair];
      reach_seen[pair] = 0;
      if (pair_is_cand(pi, krem) && seen != pi.total) atomicMin(status, STATUS_INTERNAL);
    }
  } else {
    const uint2 s = state[pair];
    prefix = s.x;
    krem = s.y;
  }
  find_digit<(NW * 32)>(sh, nb, krem, sh_scan, res);
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
__global__ void __launch_bounds__(SEL_THREADS, 8)
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
    const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + SEL_THREADS * 4 - 1) / (SEL_THREADS * 4));
    const float* a = acc + static_cast<uint64_t>(w) * N;
    for (uint32_t it = 0; it < n_iter; ++it) {
      const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * SEL_THREADS + threadIdx.x) * 4;
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
// NW warps per CTA (4: fits beside the streaming pass; 8: half the latency).
template <bool VEC, int NW>
__global__ void __launch_bounds__(NW * 32, 512 / (NW * 32) * 2)
    k_write(const float* __restrict__ acc, const float* __restrict__ weights, const Chunk* __restrict__ chunks,
            const Tile* __restrict__ tiles, const LayerDesc* __restrict__ layers, const PairInfo* __restrict__ info,
            const uint32_t* __restrict__ cand_key, const float* __restrict__ cand_val,
            const uint16_t* __restrict__ cand_idx, const uint32_t* __restrict__ cand_cnt,
            const uint2* __restrict__ state, const uint2* __restrict__ chunk_cnt, uint32_t* __restrict__ sel_idx,
            float* __restrict__ sel_val, uint32_t* __restrict__ sel_slot, const uint32_t* __restrict__ chunk_sfx,
            int* __restrict__ status, float eps, uint64_t N, uint64_t K, int W, uint32_t n_chunks, int leader,
            WorkerSel ws, const int32_t* __restrict__ layer_leader, const uint32_t* __restrict__ chunk_ids) {
  __shared__ uint32_t sh_warp[NW];
  __shared__ uint32_t sh_base[2];
  const uint32_t ci = chunk_ids != nullptr ? chunk_ids[blockIdx.x] : blockIdx.x;
  const Chunk c = chunks[ci];
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
    for (uint32_t j = c.first_chunk_of_layer + threadIdx.x; j < ci; j += (NW * 32)) {
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

  const bool is_leader = w == (layer_leader != nullptr ? layer_leader[c.layer] : leader);
  if (pair_is_cand(info[pair], L.k)) {
    // warp order is index order: count per warp, prefix over the warps, then every warp writes its
    // tiles front to back, ranking the entries of a slot with one warp scan per 128 entries
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t my_gt = 0, my_eq = 0;
    for_each_candidate<NW>(c, w, W, cand_cnt, cand_key, [&](uint32_t key) {
      my_gt += key > T ? 1u : 0u;
      my_eq += key == T ? 1u : 0u;
    });
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      my_gt += __shfl_xor_sync(0xffffffffu, my_gt, d);
      my_eq += __shfl_xor_sync(0xffffffffu, my_eq, d);
    }
    __shared__ uint32_t sh_wg[NW], sh_we[NW];
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
    const uint32_t t_begin = min(c.n_tiles, warp * tiles_per_warp<NW>(c));
    const uint32_t t_end = min(c.n_tiles, t_begin + tiles_per_warp<NW>(c));
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
            // the listed element lies inside its layer; the slot entry is one of the stored ones
            IWP_DBG_CHECK(status, tile_base + ii[u] >= L.off && tile_base + ii[u] - L.off < L.n && j + u < cnt);
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
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + (NW * 32) * 4 - 1) / ((NW * 32) * 4));
  const float* a = acc + static_cast<uint64_t>(w) * N;
  for (uint32_t it = 0; it < n_iter; ++it) {
    const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * (NW * 32) + threadIdx.x) * 4;
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
    const uint32_t ex = block_excl_scan<NW>(packed, sh_warp, total);
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
            int* __restrict__ status, float eps, uint64_t N, uint64_t K, int leader, int only_worker, float momentum,
            const int32_t* __restrict__ layer_leader) {
  extern __shared__ uint32_t keys[];
  __shared__ uint32_t hist[NBINS];
  __shared__ uint32_t sh_scan[THREADS];
  __shared__ uint32_t sh_warp[WARPS];
  __shared__ uint32_t res[4];
  const LayerDesc L = layers[small_ids[blockIdx.x]];
  const int w = blockIdx.y;
  const int tid = threadIdx.x;
  if (layer_leader != nullptr) leader = layer_leader[small_ids[blockIdx.x]];
  const uint32_t n = L.n;
  float* a = acc + static_cast<uint64_t>(w) * N + L.off;
  const float* g = grads + static_cast<uint64_t>(w) * N + L.off;
  const float* wt = weights + L.off;
  // step (a)+(b): four elements per thread and trip, all loads issued before any is used (one CTA walks the
  // whole layer, so memory-level parallelism has to come from here)
  constexpr int U = 4;
  for (uint32_t i0 = 0; i0 < n; i0 += THREADS * U) {
    float av[U], gv[U], wv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t i = i0 + u * THREADS + tid;
      av[u] = gv[u] = 0.f;
      wv[u] = 1.f;
      if (i < n) {
        av[u] = a[i];
        gv[u] = __ldcs(g + i);
        wv[u] = wt[i];
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t i = i0 + u * THREADS + tid;
      if (i < n) {
        const float v = accumulate(av[u], gv[u], momentum);
        a[i] = v;
        keys[i] = imp_key(v, wv[u], eps);
        if (w == 0) update[L.off + i] = 0.0f;
      }
    }
  }
  if (only_worker >= 0 && w != only_worker) return;  // only the chosen node selects: steps (a), (b) were this worker's part
  __syncthreads();
  uint32_t T, r;
  if (!smem_radix_select(keys, n, L.k, hist, sh_scan, res, T, r)) {
    if (tid == 0) atomicMin(status, STATUS_INTERNAL);
    return;
  }
  uint32_t* out_i = sel_idx + static_cast<uint64_t>(w) * K + L.koff;
  float* out_v = sel_val + static_cast<uint64_t>(w) * K + L.koff;
  // ordered compaction: warp q owns the q-th contiguous stretch of the layer (a multiple of 32 elements), counts
  // its keys above / at the threshold, and after one prefix over the warps ranks them 32 at a time by ballots
  const int lane = tid & 31, warp = tid >> 5;
  const uint32_t per_warp = (((n + WARPS - 1) / WARPS) + 31u) & ~31u;
  const uint32_t wb = min(n, warp * per_warp), we = min(n, wb + per_warp);
  uint32_t my_gt = 0, my_eq = 0;
  for (uint32_t i = wb + lane; i < we; i += 32) {
    const uint32_t key = keys[i];
    my_gt += key > T ? 1u : 0u;
    my_eq += key == T ? 1u : 0u;
  }
  my_gt = __reduce_add_sync(0xffffffffu, my_gt);
  my_eq = __reduce_add_sync(0xffffffffu, my_eq);
  __shared__ uint32_t sh_we[WARPS];
  if (lane == 0) {
    sh_warp[warp] = my_gt;
    sh_we[warp] = my_eq;
  }
  __syncthreads();
  uint32_t g_before = 0, q_before = 0;
  for (int q = 0; q < warp; ++q) {
    g_before += sh_warp[q];
    q_before += sh_we[q];
  }
  if ((my_gt | my_eq) == 0) return;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (uint32_t i0 = wb; i0 < we; i0 += 32) {
    const uint32_t i = i0 + lane;
    const uint32_t key = i < we ? keys[i] : 0u;
    const bool isg = i < we && key > T, ise = i < we && key == T;
    const uint32_t bg = __ballot_sync(0xffffffffu, isg), be = __ballot_sync(0xffffffffu, ise);
    const uint32_t gb = g_before + __popc(bg & lt_mask), qb = q_before + __popc(be & lt_mask);
    if (isg || (ise && qb < r)) {
      const uint32_t pos = gb + (qb < r ? qb : r);
      if (pos < L.k) {
        out_i[pos] = L.off + i;
        out_v[pos] = a[i];
        if (w == leader) sel_slot[L.koff + pos] = REF_NONE;
      } else {
        atomicMin(status, STATUS_INTERNAL);
      }
    }
    g_before += __popc(bg);
    q_before += __popc(be);
  }
}

}  // namespace iwp

namespace iwp {

// ---------------------------------------------------------------------------------------
// single-read path, steps (c)+(d) in ONE launch for layers of at most PAIR_MAX_TILES tiles: a thread-block
// CLUSTER of PAIR_CLUSTER CTAs per (layer, worker) pair.  Each CTA takes a contiguous share of the pair's tiles,
// copies their candidate keys into shared memory, and the cluster runs the three digit passes of the exact radix
// select on them - local shared-memory histograms, merged through distributed shared memory - and writes the
// ordered list, every CTA its own part at an offset taken from the other CTAs' counts.  It replaces seven
// dependent launches (three histogram passes with their digit decisions, then the compaction) whose CTAs mostly
// wait on each other.  CTAs of a cluster meet only at cluster.sync(), a hardware barrier: nothing spins.
// A pair whose guess failed (fewer than k elements reached it, or a slot overflowed) is selected by the same
// cluster from the residuals and weights themselves: exact, slower, and rare.
// grid = (pair layers * PAIR_CLUSTER, covered workers); THREADS threads; dynamic shared memory =
// 4 * PAIR_KEYS_SMEM bytes.
// ---------------------------------------------------------------------------------------
constexpr int PAIR_CLUSTER = 8;
constexpr uint32_t PAIR_KEYS_SMEM = 16384;  // candidate keys a CTA keeps in shared memory (the rest is re-read)
constexpr uint32_t PAIR_CTA_TILES = (PAIR_MAX_TILES + PAIR_CLUSTER - 1) / PAIR_CLUSTER;

// Merges the CTAs' local histograms and leaves the sum in every CTA's `hist`.  CTA r adds up bins
// [r * THREADS, (r + 1) * THREADS) of all CTAs into CTA 0's `merged`; after the barrier everybody copies it.
// Contains two cluster barriers and one block barrier.
__device__ __forceinline__ void cluster_merge_hist(cooperative_groups::cluster_group& cluster, uint32_t* hist,
                                                   uint32_t* merged, int nb) {
  static_assert(NBINS == PAIR_CLUSTER * THREADS, "one bin per thread and CTA of the cluster");
  const unsigned cr = cluster.block_rank();
  cluster.sync();  // every local histogram is complete
  const int b = static_cast<int>(cr) * THREADS + static_cast<int>(threadIdx.x);
  if (b < nb) {
    uint32_t sum = 0;
#pragma unroll
    for (int q = 0; q < PAIR_CLUSTER; ++q) sum += cluster.map_shared_rank(hist, q)[b];
    cluster.map_shared_rank(merged, 0)[b] = sum;
  }
  cluster.sync();  // the merged histogram is complete, nobody reads a local one any more
  const uint32_t* src = cluster.map_shared_rank(merged, 0);
  for (int q = threadIdx.x; q < nb; q += THREADS) hist[q] = src[q];
  __syncthreads();
}

template <bool VEC>
__global__ void __cluster_dims__(PAIR_CLUSTER, 1, 1) __launch_bounds__(THREADS)
    k_select_pair(const float* __restrict__ acc, const float* __restrict__ weights, const Tile* __restrict__ tiles,
                  const LayerDesc* __restrict__ layers, const uint32_t* __restrict__ pair_layer_ids,
                  const PairInfo* __restrict__ info, const uint32_t* __restrict__ cand_key,
                  const float* __restrict__ cand_val, const uint16_t* __restrict__ cand_idx,
                  const uint32_t* __restrict__ cand_cnt, uint2* __restrict__ state, uint32_t* __restrict__ sel_idx,
                  float* __restrict__ sel_val, uint32_t* __restrict__ sel_slot, int* __restrict__ status, float eps,
                  uint64_t N, uint64_t K, int W, int leader, WorkerSel ws, const int32_t* __restrict__ layer_leader) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned cr = cluster.block_rank();
  extern __shared__ uint32_t keys[];  // this CTA's first PAIR_KEYS_SMEM candidate keys, in slot order
  __shared__ uint32_t hist[NBINS];
  __shared__ uint32_t merged[NBINS];                // CTA 0's copy is the cluster's
  __shared__ uint32_t x_cnt[PAIR_CLUSTER][2];       // CTA 0's copy: every CTA's (#keys > T, #keys == T)
  __shared__ uint32_t x_reach;                      // CTA 0's copy: stored entries that reach the guess
  __shared__ uint32_t sh_scan[WARPS];
  __shared__ uint32_t res[4];
  __shared__ uint32_t tile_off[PAIR_CTA_TILES + 1];  // exclusive prefix of this CTA's tiles' stored candidate counts
  __shared__ uint32_t sh_wg[WARPS], sh_we[WARPS];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t layer_id = pair_layer_ids[blockIdx.x / PAIR_CLUSTER];
  const LayerDesc L = layers[layer_id];
  const int w = sel_worker(ws, static_cast<int>(blockIdx.y));
  const uint32_t pair = static_cast<uint32_t>(L.large_index) * W + w;
  const PairInfo pi = info[pair];
  const bool is_leader = w == (layer_leader != nullptr ? layer_leader[layer_id] : leader);
  const bool cand = pair_is_cand(pi, L.k);
  uint32_t* out_i = sel_idx + static_cast<uint64_t>(w) * K + L.koff;
  float* out_v = sel_val + static_cast<uint64_t>(w) * K + L.koff;
  if (tid == 0) x_reach = 0;
  cluster.sync();  // every CTA of the cluster runs and has cleared what others add to

  // this CTA's share: tiles [t0, t1) of the pair, or (guess failed) elements [lo, hi) of the layer
  const uint32_t per = (L.n_tiles + PAIR_CLUSTER - 1) / PAIR_CLUSTER;
  const uint32_t t0 = min(L.n_tiles, cr * per), t1 = min(L.n_tiles, t0 + per), nt = t1 - t0;
  const uint64_t share = ((static_cast<uint64_t>(L.n) + PAIR_CLUSTER - 1) / PAIR_CLUSTER + 3) & ~3ull;
  const uint64_t lo = min(static_cast<uint64_t>(L.off) + L.n, L.off + cr * share), hi = min(static_cast<uint64_t>(L.off) + L.n, lo + share);
  const uint64_t s0 = lo & ~3ull;
  const uint32_t n_iter = static_cast<uint32_t>((hi - s0 + THREADS * 4 - 1) / (THREADS * 4));
  const float* a = acc + static_cast<uint64_t>(w) * N;
  auto slot_of = [&](uint32_t t) { return (static_cast<uint64_t>(L.first_tile + t0 + t) * W + w) * CAND_CAP; };
  uint32_t total = 0;  // stored candidates of this CTA's tiles

  if (cand) {
    for (uint32_t t = tid; t < nt; t += THREADS)
      tile_off[t + 1] = min(cand_cnt[static_cast<uint64_t>(L.first_tile + t0 + t) * W + w], CAND_CAP);
    if (tid == 0) tile_off[0] = 0;
    __syncthreads();
    if (warp == 0) {  // inclusive scan in place, 32 tiles at a time
      uint32_t run = 0;
      for (uint32_t b = 0; b < nt; b += 32) {
        const uint32_t t = b + lane;
        const uint32_t v = t < nt ? tile_off[t + 1] : 0u;
        const uint32_t incl = warp_incl_scan(v);
        if (t < nt) tile_off[t + 1] = run + incl;
        run += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
    __syncthreads();
    total = tile_off[nt];
    // keys into shared memory, four tiles per warp and trip with all loads issued first
    for (uint32_t tb = warp * 4; tb < nt; tb += WARPS * 4) {
      uint4 k4[4];
      uint32_t cnt[4], p0[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t t = tb + q;
        p0[q] = t < nt ? tile_off[t] : 0u;
        cnt[q] = t < nt ? tile_off[t + 1] - p0[q] : 0u;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)  // slots are zero-padded to groups of four entries
        k4[q] = (static_cast<uint32_t>(lane) * 4 < cnt[q]) ? reinterpret_cast<const uint4*>(cand_key + slot_of(tb + q))[lane]
                                                           : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t kk[4] = {k4[q].x, k4[q].y, k4[q].z, k4[q].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t j = lane * 4 + u;
          if (j < cnt[q] && p0[q] + j < PAIR_KEYS_SMEM) keys[p0[q] + j] = kk[u];
        }
        for (uint32_t j = 128 + lane; j < cnt[q]; j += 32)  // the rare slot with more than 128 entries
          if (p0[q] + j < PAIR_KEYS_SMEM) keys[p0[q] + j] = cand_key[slot_of(tb + q) + j];
      }
    }
    __syncthreads();
  }
  // f(key) over this CTA's keys: the cached ones flat out of shared memory, the rest (a CTA whose tiles hold more
  // than PAIR_KEYS_SMEM candidates) tile by tile through the L2; or, guess failed, over its share of the layer
  auto for_each_key = [&](auto&& f) {
    if (cand) {
      const uint32_t cached = min(total, PAIR_KEYS_SMEM);
      for (uint32_t p = tid; p < cached; p += THREADS) f(keys[p]);
      if (total > PAIR_KEYS_SMEM) {
        for (uint32_t t = warp; t < nt; t += WARPS) {
          if (tile_off[t + 1] <= PAIR_KEYS_SMEM) continue;
          const uint32_t first = tile_off[t] >= PAIR_KEYS_SMEM ? 0u : PAIR_KEYS_SMEM - tile_off[t];
          const uint32_t cnt = tile_off[t + 1] - tile_off[t];
          for (uint32_t j = first + lane; j < cnt; j += 32) f(cand_key[slot_of(t) + j]);
        }
      }
    } else {
      for (uint32_t it = 0; it < n_iter; ++it) {
        const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + tid) * 4;
        float av[4], wv[4];
        load4<VEC>(a, e0, lo, hi, av);
        load4<VEC>(weights, e0, lo, hi, wv);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (e0 + q >= lo && e0 + q < hi) f(imp_key(av[q], wv[q], eps));
      }
    }
  };

  // three digit passes
  uint32_t prefix = 0, krem = L.k;
#pragma unroll 1
  for (int pass = 0; pass < N_PASSES; ++pass) {
    const int shift = pass_shift(pass), nb = pass_bins(pass);
    const int prev_shift = pass == 0 ? 31 : pass_shift(pass - 1);
    const uint32_t want = prefix >> prev_shift;
    for (int b = tid; b < NBINS; b += THREADS) hist[b] = 0;
    __syncthreads();
    uint32_t ge = 0;
    for_each_key([&](uint32_t key) {
      if ((key >> prev_shift) == want) atomicAdd(&hist[(key >> shift) & (nb - 1)], 1u);  // pass 0: bit 31 is 0 == want
      ge += key >= pi.guess ? 1u : 0u;
    });
    if (pass == 0 && cand) {  // the stored entries that reach the guess, re-counted (conservation check)
      ge = __reduce_add_sync(0xffffffffu, ge);
      if (lane == 0 && ge) atomicAdd(cluster.map_shared_rank(&x_reach, 0), ge);
    }
    __syncthreads();
    cluster_merge_hist(cluster, hist, merged, nb);
    if (pass == 0 && cand && cr == 0 && tid == 0 && x_reach != pi.total) atomicMin(status, STATUS_INTERNAL);
    find_digit(hist, nb, krem, sh_scan, res);
    const bool found = res[2] != 0;
    const uint32_t d = res[0], kr = res[1];
    __syncthreads();
    if (!found) {  // the same in every CTA of the cluster
      if (cr == 0 && tid == 0) {
        atomicMin(status, STATUS_INTERNAL);
        state[pair] = make_uint2(0xffffffffu, 0u);
      }
      cluster.sync();  // nobody leaves while its shared memory may still be read
      return;
    }
    prefix |= d << shift;
    krem = kr;
  }
  const uint32_t T = prefix, r = krem;
  if (cr == 0 && tid == 0) state[pair] = make_uint2(T, r);

  // list offset of this CTA's part: the counts of the CTAs in front of it
  {
    uint32_t gt = 0, eq = 0;
    for_each_key([&](uint32_t key) {
      gt += key > T ? 1u : 0u;
      eq += key == T ? 1u : 0u;
    });
    gt = __reduce_add_sync(0xffffffffu, gt);
    eq = __reduce_add_sync(0xffffffffu, eq);
    if (lane == 0) {
      sh_wg[warp] = gt;
      sh_we[warp] = eq;
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t g = 0, e = 0;
      for (int q = 0; q < WARPS; ++q) {
        g += sh_wg[q];
        e += sh_we[q];
      }
      uint32_t* dst = cluster.map_shared_rank(&x_cnt[0][0], 0);
      dst[2 * cr] = g;
      dst[2 * cr + 1] = e;
    }
  }
  cluster.sync();
  uint32_t run_gt = 0, run_eq = 0;
  {
    const uint32_t* src = cluster.map_shared_rank(&x_cnt[0][0], 0);
    for (unsigned q = 0; q < cr; ++q) {
      run_gt += src[2 * q];
      run_eq += src[2 * q + 1];
    }
  }
  cluster.sync();  // the last remote read is done: from here on every CTA is on its own

  if (!cand) {  // ordered compaction of this CTA's share of the layer
    for (uint32_t it = 0; it < n_iter; ++it) {
      const uint64_t e0 = s0 + (static_cast<uint64_t>(it) * THREADS + tid) * 4;
      float av[4], wv[4];
      load4<VEC>(a, e0, lo, hi, av);
      load4<VEC>(weights, e0, lo, hi, wv);
      uint32_t fg = 0, fe = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint64_t e = e0 + q;
        const bool in = e >= lo && e < hi;
        const uint32_t key = imp_key(av[q], wv[q], eps);
        fg |= (in && key > T) ? (1u << q) : 0u;
        fe |= (in && key == T) ? (1u << q) : 0u;
      }
      uint32_t tot;
      const uint32_t packed = static_cast<uint32_t>(__popc(fg)) | (static_cast<uint32_t>(__popc(fe)) << 16);
      const uint32_t ex = block_excl_scan(packed, sh_scan, tot);
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
      run_gt += tot & 0xffffu;
      run_eq += tot >> 16;
    }
    return;
  }

  // ordered compaction from the slots: batches of WARPS * 4 consecutive tiles, warp q the q-th group of four, so
  // that warp order is index order.  Each lane takes four consecutive entries of a slot; keys, values and offsets
  // of the warp's four tiles are all requested before any is used; ranks come from one warp scan per 128 entries.
  for (uint32_t tb0 = 0; tb0 < nt; tb0 += WARPS * 4) {
    const uint32_t t_begin = min(nt, tb0 + warp * 4), t_end = min(nt, t_begin + 4);
    uint32_t cnt[4];
    uint4 k4[4];
    float4 v4[4];
    uint2 i2[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) cnt[q] = (t_begin + q < t_end) ? tile_off[t_begin + q + 1] - tile_off[t_begin + q] : 0u;
#pragma unroll
    for (int q = 0; q < 4; ++q) {  // slots are zero-padded to groups of four entries; entries past the count are masked
      const bool has = static_cast<uint32_t>(lane) * 4 < cnt[q];
      const uint64_t slot = slot_of(t_begin + q);
      k4[q] = has ? reinterpret_cast<const uint4*>(cand_key + slot)[lane] : make_uint4(0u, 0u, 0u, 0u);
      v4[q] = has ? reinterpret_cast<const float4*>(cand_val + slot)[lane] : make_float4(0.f, 0.f, 0.f, 0.f);
      i2[q] = has ? reinterpret_cast<const uint2*>(cand_idx + slot)[lane] : make_uint2(0u, 0u);
    }
    // flags of a lane's four entries of one group of 128
    auto flags = [&](uint32_t cnt_t, uint32_t j0, uint4 k, uint32_t& fg, uint32_t& fe) {
      const uint32_t j = j0 + lane * 4;
      const uint32_t kk[4] = {k.x, k.y, k.z, k.w};
      fg = fe = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const bool in = j + u < cnt_t;
        fg |= (in && kk[u] > T) ? (1u << u) : 0u;
        fe |= (in && kk[u] == T) ? (1u << u) : 0u;
      }
    };
    auto group = [&](uint32_t t, uint32_t g) {  // group g of 128 entries of tile t, beyond the preloaded first one
      const uint64_t slot = slot_of(t);
      return reinterpret_cast<const uint4*>(cand_key + slot)[g * 32 + lane];
    };
    uint32_t my_gt = 0, my_eq = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t fg, fe;
      flags(cnt[q], 0, k4[q], fg, fe);
      my_gt += __popc(fg);
      my_eq += __popc(fe);
      for (uint32_t j0 = 128; j0 < cnt[q]; j0 += 128) {  // the rare slot with more than 128 entries
        flags(cnt[q], j0, (j0 + lane * 4 < cnt[q]) ? group(t_begin + q, j0 >> 7) : make_uint4(0u, 0u, 0u, 0u), fg, fe);
        my_gt += __popc(fg);
        my_eq += __popc(fe);
      }
    }
    my_gt = __reduce_add_sync(0xffffffffu, my_gt);
    my_eq = __reduce_add_sync(0xffffffffu, my_eq);
    __syncthreads();  // the previous batch has read the per-warp counts
    if (lane == 0) {
      sh_wg[warp] = my_gt;
      sh_we[warp] = my_eq;
    }
    __syncthreads();
    uint32_t g_before = run_gt, q_before = run_eq, tot_g = 0, tot_e = 0;
#pragma unroll
    for (int q = 0; q < WARPS; ++q) {
      const uint32_t g = sh_wg[q], e = sh_we[q];
      if (q < warp) {
        g_before += g;
        q_before += e;
      }
      tot_g += g;
      tot_e += e;
    }
    run_gt += tot_g;
    run_eq += tot_e;
    if ((my_gt | my_eq) == 0) continue;  // nothing of this warp's tiles is selected
    auto emit = [&](uint32_t t, uint32_t cnt_t, uint32_t j0, uint4 k, float4 vals, uint2 offs) {
      const uint32_t j = j0 + lane * 4;
      const uint32_t tile = L.first_tile + t0 + t;
      const uint32_t tile_base = tiles[tile].a & ~(TILE - 1u);
      uint32_t fg, fe;
      flags(cnt_t, j0, k, fg, fe);
      const uint32_t packed = static_cast<uint32_t>(__popc(fg)) | (static_cast<uint32_t>(__popc(fe)) << 16);
      const uint32_t incl = warp_incl_scan(packed);
      const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
      uint32_t gb = g_before + ((incl - packed) & 0xffffu), qb = q_before + ((incl - packed) >> 16);
      if (fg | fe) {
        const float vv[4] = {vals.x, vals.y, vals.z, vals.w};
        const uint32_t ii[4] = {offs.x & 0xffffu, offs.x >> 16, offs.y & 0xffffu, offs.y >> 16};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool isg = (fg >> u) & 1u, ise = (fe >> u) & 1u;
          if (isg || (ise && qb < r)) {
            const uint32_t pos = gb + (qb < r ? qb : r);
            IWP_DBG_CHECK(status, tile_base + ii[u] >= L.off && tile_base + ii[u] - L.off < L.n);
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
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (cnt[q] == 0) continue;
      const uint32_t t = t_begin + q;
      emit(t, cnt[q], 0, k4[q], v4[q], i2[q]);
      for (uint32_t j0 = 128; j0 < cnt[q]; j0 += 128) {
        const bool has = j0 + lane * 4 < cnt[q];
        const uint64_t slot = slot_of(t);
        const uint32_t g = (j0 >> 2) + lane;
        emit(t, cnt[q], j0, has ? reinterpret_cast<const uint4*>(cand_key + slot)[g] : make_uint4(0u, 0u, 0u, 0u),
             has ? reinterpret_cast<const float4*>(cand_val + slot)[g] : make_float4(0.f, 0.f, 0.f, 0.f),
             has ? reinterpret_cast<const uint2*>(cand_idx + slot)[g] : make_uint2(0u, 0u));
      }
    }
  }
}

}  // namespace iwp

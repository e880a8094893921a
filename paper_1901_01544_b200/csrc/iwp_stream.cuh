// Steps (a)+(b) of the pruning step: the plain accumulate pass and the single-read streaming pass (accumulate,
// importance, candidate emission, side values).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_device.cuh"

namespace iwp {

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
// roundings of gm * den and the one of the quotient are each below 2^-23 relative).  Only the
// elements that pass (about 2 % at a keep ratio of 1/64) get the exact IEEE quotient: each lane
// handles its own, in index order, and stores key, value and offset at the element's rank in the
// slot.  Keeping the few entries that fall just short of the guess is harmless: whenever at least k
// elements of the layer reach the guess, the k best of this superset are the k best of the layer.
// The argument needs normal products, so the pre-test is disabled (gm = 0: everything passes) for
// tiny guesses or eps.
// ---------------------------------------------------------------------------------------


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
// packed 8 bits per round (a round stages at most 128 elements, so a field never carries).  The
// sum over the earlier rounds reaches 384 and is therefore taken in a full register: a byte-wise
// dot product of the totals with a 0/1 selector of the rounds below this one.
__device__ __forceinline__ uint32_t staged_position(uint32_t mask, uint32_t ex, uint32_t tt, uint32_t b) {
  const uint32_t round = b >> 2;
  const uint32_t earlier = 0x00010101u >> (8u * (3u - round));  // byte r is 1 for every round r < round
  const uint32_t rounds_before = __dp4a(tt, earlier, 0u);
  return rounds_before + ((ex >> (8u * round)) & 0xFFu) + __popc((mask >> (b & ~3u)) & ((1u << (b & 3u)) - 1u));
}

template <bool VEC, bool LEADER>
__global__ void __launch_bounds__(THREADS, 3)
    k_stream(const float* __restrict__ grads, const float* __restrict__ weights, float* __restrict__ acc,
             float* __restrict__ update, const Tile* __restrict__ tiles, PairInfo* __restrict__ info,
             const uint2* __restrict__ guess_tab, uint32_t* __restrict__ cand_key, float* __restrict__ cand_val,
             uint16_t* __restrict__ cand_idx, uint32_t* __restrict__ cand_cnt, float* __restrict__ side_val,
             uint2* __restrict__ lead_lane, uint32_t* __restrict__ lead_tot, const uint32_t* __restrict__ zmask,
             float eps, uint64_t N, int W, int leader, uint32_t n_tiles, int worker_groups, float momentum,
             int* __restrict__ status, const int32_t* __restrict__ layer_leader) {
  constexpr int ROUNDS = SEG_ELEMS / 128;  // 128-bit slots per lane and iteration = 4
  __shared__ __align__(16) float r_val[WARPS][SEG_ELEMS];  // results of the iteration, for run-time indexing
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t tile_id;
  int wi = 0;
  if (LEADER) {  // eight tiles of the leader per CTA
    tile_id = blockIdx.x * WARPS + warp;
    if (tile_id >= n_tiles) return;
  } else {  // up to eight of the other workers of one tile per CTA: the tile's weights come through L1
    tile_id = blockIdx.x / worker_groups;
    wi = static_cast<int>(blockIdx.x % worker_groups) * static_cast<int>(blockDim.x >> 5) + warp;
    if (wi >= W - 1) return;
  }
  const Tile t = tiles[tile_id];
  // the chosen node: one per step, or (option "per_layer_leaders") the one drawn for this tile's layer
  if (layer_leader != nullptr) leader = layer_leader[t.layer];
  const int w = LEADER ? leader : (wi < leader ? wi : wi + 1);
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
  float* res = r_val[warp] + lane * 4;
  uint32_t count = 0;    // entries appended to the slot so far (the same in every lane)
  uint32_t reached = 0;  // of those, how many reach the guess exactly (this lane's share until the final reduction)
  uint32_t dbg_passed = 0;  // debug build: elements of this lane that passed the pre-test (count conservation)
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
    IWP_DBG_CHECK(status, (seg >> 9) < (N >> 9) + 2);  // the segment's zero-mask fields exist
    zm_next = reinterpret_cast<const uint16_t*>(zmask)[(seg >> 9) * 32 + lane];
    if (!LEADER) {  // the leader's record for this segment: (mask | count << 16, lane prefix), round totals
      const uint64_t sigma = static_cast<uint64_t>(tile_id) * SEGS_PER_TILE + it;
      IWP_DBG_CHECK(status, it < SEGS_PER_TILE && tile_id < n_tiles);
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
        IWP_DBG_CHECK(status, pos < TILE && b < 16u);  // a rank inside the chosen node's tile, a bit of its 16-bit mask
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
      // every lane takes its own elements that passed the pre-test: exact quotient, then key, value and
      // offset straight to the slot at the element's rank (the ranks of a warp's elements are consecutive,
      // so the stores of one trip fall into a few sectors)
      for (uint32_t mm = m; mm; mm &= mm - 1) {
        const uint32_t b = __ffs(mm) - 1;
        const uint32_t pos = count + staged_position(m, excl, tot, b);
        const uint32_t off = (b >> 2) * 128 + (b & 3u);
        // ranks inside an iteration stay below the iteration's total, and the element is one of the tile's
        IWP_DBG_CHECK(status, pos - count < (tot & 0xFFu) + ((tot >> 8) & 0xFFu) + ((tot >> 16) & 0xFFu) + (tot >> 24));
        IWP_DBG_CHECK(status, first + off >= lo && first + off < hi);
        if (DEBUG_CHECKS) ++dbg_passed;
        const float v = res[off];
        const uint32_t key = imp_key_den(v, imp_den(weights[first + off], eps));  // weight re-read through L1
        reached += (key >= guess) ? 1u : 0u;
        if (pos < CAND_CAP) {
          st_keep_u32(cand_key + slot + pos, key, keep);
          st_keep_f32(cand_val + slot + pos, v, keep);
          st_keep_u16(cand_idx + slot + pos, static_cast<uint16_t>(static_cast<uint32_t>(first - base) + off), keep);
        }
      }
      count += (tot & 0xFFu) + ((tot >> 8) & 0xFFu) + ((tot >> 16) & 0xFFu) + (tot >> 24);
    }
  }
  reached = __reduce_add_sync(0xffffffffu, reached);
  if (DEBUG_CHECKS) {  // every element that passed the pre-test was given exactly one rank
    dbg_passed = __reduce_add_sync(0xffffffffu, dbg_passed);
    IWP_DBG_CHECK(status, dbg_passed == count);
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
    if (count > CAND_CAP) atomicOr(&info[pair].flags, 1u);  // more candidates than the slot holds: exact fallback
  }
}

}  // namespace iwp

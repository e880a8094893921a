// Steps (e)-(g) of the pruning step: the reduction at the chosen node's index set in its variants (gather,
// side values, union of several chosen nodes, workers spread over contexts), the zero-mask flush, the copies
// kept for late selects and the byte mask accessor.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_device.cuh"
#include "iwp_stream.cuh"

namespace iwp {

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
// worker order and scatters the sum - and every later entry with the same element returns at once.  The
// marks stay set and are the zeroing: the next streaming pass (or the flush before anything else looks at
// the residuals) takes a marked residual as +0, which saves W scattered 4-byte stores per element here.
// Only elements of one-CTA layers, which no streaming pass visits, are zeroed on the spot (their mark is
// then redundant).
__global__ void __launch_bounds__(THREADS)
    k_union_sum_scatter(const uint32_t* __restrict__ sel_idx, float* __restrict__ acc, float* __restrict__ update,
                        uint32_t* __restrict__ seen, uint64_t N, uint64_t K, int W, LeaderSet ls,
                        const LayerDesc* __restrict__ layers, uint32_t n_layers, int first_node) {
  // first_node = 1: r_1's list was already reduced from the side values of the streaming pass (k_sum_scatter,
  // which marked every element it owns); this launch covers the lists of r_2 .. r_n
  const uint64_t q = static_cast<uint64_t>(first_node) * K + static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
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
  update[i] = __fadd_rn(0.0f, s);
  uint32_t lo = 0, hi = n_layers - 1;  // the layer whose list segment holds this entry
  const uint64_t e = q % K;
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    if (layers[mid].koff <= e) lo = mid; else hi = mid - 1;
  }
  if (layers[lo].large_index < 0)
    for (int w = 0; w < W; ++w) p[static_cast<uint64_t>(w) * N] = 0.0f;
}

// Steps (e)-(g) when every layer has its own chosen node (Algorithm 1 draws the node inside its loop over
// layers): entry j of the index set lies in the list segment of one layer and comes from that layer's
// node's list.  One thread per entry: find the layer (binary search over the segment offsets), draw its
// node, then gather, sum in ascending worker order, scatter and zero.  With dst != nullptr the kernel only
// marks the index set in a byte mask (accessor).
__global__ void __launch_bounds__(THREADS)
    k_layer_leader_sum_scatter(const uint32_t* __restrict__ sel_idx, const LayerDesc* __restrict__ layers, uint32_t n_layers,
                               float* __restrict__ acc, float* __restrict__ update, uint8_t* __restrict__ dst, uint64_t N,
                               uint64_t K, int W, uint64_t seed, uint64_t step) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= K) return;
  uint32_t lo = 0, hi = n_layers - 1;  // last layer whose segment starts at or before j
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    if (layers[mid].koff <= j) lo = mid; else hi = mid - 1;
  }
  const int r = layer_leader_at(seed, step, lo, W);
  const uint64_t i = sel_idx[static_cast<uint64_t>(r) * K + j];
  if (dst != nullptr) {
    dst[i] = 1;
    return;
  }
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
// context's own residuals are zeroed there: by a mark in the zero mask, which the next streaming pass applies
// while it reads the residuals anyway (instead of W_local scattered 4-byte stores per entry); elements of
// one-CTA layers, which no streaming pass visits, are zeroed on the spot.  One thread per entry.
__global__ void __launch_bounds__(THREADS)
    k_shard_apply(const uint32_t* __restrict__ idx, const float* __restrict__ vals_all, float* __restrict__ acc,
                  float* __restrict__ update, uint32_t* __restrict__ zmask, const LayerDesc* __restrict__ layers,
                  uint32_t n_layers, uint64_t N, uint64_t n, int W_total, int W_local, int* __restrict__ status) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= n) return;
  const uint64_t i = idx[j];
  if (i >= N) {  // not an element of this job: reported, nothing written
    atomicMin(status, STATUS_INTERNAL);
    return;
  }
  float s = vals_all[j];
  for (int w = 1; w < W_total; ++w) s = __fadd_rn(s, vals_all[static_cast<uint64_t>(w) * n + j]);
  update[i] = __fadd_rn(0.0f, s);
  uint32_t lo = 0, hi = n_layers - 1;  // the layer that holds element i
  while (lo < hi) {
    const uint32_t mid = (lo + hi + 1) >> 1;
    if (layers[mid].off <= i) lo = mid; else hi = mid - 1;
  }
  if (layers[lo].large_index < 0) {
    for (int w = 0; w < W_local; ++w) acc[static_cast<uint64_t>(w) * N + i] = 0.0f;
  } else {
    atomicOr(&zmask[zmask_word(i)], zmask_bit(i));
  }
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
                  int leader, uint64_t n_slots, int* __restrict__ status, const LayerDesc* __restrict__ layers,
                  uint32_t n_layers, const int32_t* __restrict__ layer_leader, int mark_all) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= K) return;
  if (layer_leader != nullptr) {
    // one chosen node per layer: entry j lies in one layer's list segment and comes from that layer's node's list
    // (leader_idx is then the base of all W lists)
    uint32_t lo = 0, hi = n_layers - 1;  // last layer whose segment starts at or before j
    while (lo < hi) {
      const uint32_t mid = (lo + hi + 1) >> 1;
      if (layers[mid].koff <= j) lo = mid; else hi = mid - 1;
    }
    leader = layer_leader[lo];
    leader_idx += static_cast<uint64_t>(leader) * K;
  }
  const uint64_t i = leader_idx[j];
  const uint32_t ref = sel_slot[j];
  // the entry is an element of the job, and it names a position of an existing (tile, worker) slot
  IWP_DBG_CHECK(status, i < N && (ref >= REF_LAZY || (ref / CAND_CAP) * W + (W - 1) < n_slots));
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
      if (mark_all) atomicOr(&zmask[zmask_word(i)], zmask_bit(i));  // a later launch must see that it is taken
    }
  }
  update[i] = __fadd_rn(0.0f, s);
}

// Option "per_layer_leaders": the chosen node of every layer for this step, one table entry per layer.
__global__ void __launch_bounds__(THREADS)
    k_layer_leaders(int32_t* __restrict__ layer_leader, uint32_t n_layers, uint64_t seed, uint64_t step, int W) {
  const uint32_t l = blockIdx.x * THREADS + threadIdx.x;
  if (l < n_layers) layer_leader[l] = layer_leader_at(seed, step, l, W);
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

// byte mask of the index set (Algorithm 1's encode_uint8(Mask)); dst is zeroed by the caller
__global__ void __launch_bounds__(THREADS) k_mask_scatter(const uint32_t* __restrict__ leader_idx, uint8_t* __restrict__ dst, uint64_t K) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j < K) dst[leader_idx[j]] = 1;
}

// The byte mask at eight elements per byte (the other reading of encode_uint8(Mask)): bit i % 8 of byte
// i / 8 is element i's mask value.  One thread per output byte.
__global__ void __launch_bounds__(THREADS) k_pack_mask(const uint8_t* __restrict__ mask, uint8_t* __restrict__ bits, uint64_t N) {
  const uint64_t b = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (b * 8 >= N) return;
  uint32_t v = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const uint64_t i = b * 8 + q;
    if (i < N && mask[i]) v |= 1u << q;
  }
  bits[b] = static_cast<uint8_t>(v);
}

}  // namespace iwp

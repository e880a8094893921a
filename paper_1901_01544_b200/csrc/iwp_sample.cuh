// Threshold guess of the single-read path: a sample of every (tiled layer, worker) pair.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_device.cuh"

namespace iwp {

// ---------------------------------------------------------------------------------------
// single-read path, threshold guess: one CTA per (tiled layer, worker) pair evaluates the
// importance the step WILL produce (acc + grad) on a strided, jittered sample of the layer and
// takes the rho-th largest as the guess.  Only a guess: the select stays exact whatever it is.
// grid = pairs; dynamic shared memory = 4 * max sample bytes.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t hash32(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
  return x;
}

constexpr int SAMPLE_THREADS = 1024;

__global__ void __launch_bounds__(SAMPLE_THREADS)
    k_sample(const float* __restrict__ grads, const float* __restrict__ weights, const float* __restrict__ acc,
             const LayerDesc* __restrict__ layers, const uint32_t* __restrict__ large_ids, PairInfo* __restrict__ info,
             uint2* __restrict__ guess_tab, const uint32_t* __restrict__ zmask, float eps, uint64_t N, int W,
             uint32_t step, int only_worker, float momentum) {
  extern __shared__ uint32_t keys[];
  __shared__ uint32_t hist[NBINS];
  __shared__ uint32_t sh_scan[SAMPLE_THREADS];
  __shared__ uint32_t res[4];
  const uint32_t pair = blockIdx.x;
  const LayerDesc L = layers[large_ids[pair / W]];
  const int w = pair % W;
  const uint32_t s = L.sample;
  if (s == 0 || (only_worker >= 0 && w != only_worker)) {  // no speculation, or a worker that makes no selection
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

}  // namespace iwp

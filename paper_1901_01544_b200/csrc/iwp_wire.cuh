// Wire formats of the index set when the workers are spread over several GPUs (Algorithm 1:
// AllGather(encode_uint8(Mask)) before the all-reduce of the masked gradients).  Two encodings travel:
// the sorted 32-bit index list (4 bytes per entry) and the mask at one bit per element (N / 8 bytes,
// bit i % 8 of byte i / 8); the sender picks the shorter.  These kernels turn one into the other.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "iwp_device.cuh"

namespace iwp {

constexpr uint32_t WIRE_WORDS_PER_THREAD = 4;
constexpr uint32_t WIRE_CHUNK_WORDS = THREADS * WIRE_WORDS_PER_THREAD;  // 32-bit mask words per CTA (32 Ki elements)

// list -> bits: one thread per entry; `words` (the mask as little-endian 32-bit words) was zeroed before.
__global__ void __launch_bounds__(THREADS)
    k_wire_pack(const uint32_t* __restrict__ idx, uint64_t n, uint32_t* __restrict__ words, uint64_t N,
                int* __restrict__ status) {
  const uint64_t j = static_cast<uint64_t>(blockIdx.x) * THREADS + threadIdx.x;
  if (j >= n) return;
  const uint32_t i = idx[j];
  if (i >= N) {  // not an element of this job: reported, never written
    atomicMin(status, STATUS_INTERNAL);
    return;
  }
  atomicOr(&words[i >> 5], 1u << (i & 31u));
}

// bits -> list, first look: set bits per chunk of WIRE_CHUNK_WORDS words.  grid = chunks.
__global__ void __launch_bounds__(THREADS)
    k_wire_count(const uint32_t* __restrict__ words, uint64_t n_words, uint32_t* __restrict__ chunk_cnt) {
  __shared__ uint32_t sh_warp[WARPS];
  const uint64_t w0 = static_cast<uint64_t>(blockIdx.x) * WIRE_CHUNK_WORDS + threadIdx.x * WIRE_WORDS_PER_THREAD;
  uint32_t c = 0;
#pragma unroll
  for (uint32_t q = 0; q < WIRE_WORDS_PER_THREAD; ++q)
    if (w0 + q < n_words) c += __popc(words[w0 + q]);
  uint32_t total;
  block_excl_scan(c, sh_warp, total);
  if (threadIdx.x == 0) chunk_cnt[blockIdx.x] = total;
}

// bits -> list, second look: ascending indices at the chunk's offset (from the scan of the chunk counts).
// Entries beyond `cap` are dropped and reported.  grid = chunks.
__global__ void __launch_bounds__(THREADS)
    k_wire_expand(const uint32_t* __restrict__ words, uint64_t n_words, const uint32_t* __restrict__ chunk_off,
                  uint32_t* __restrict__ idx, uint64_t cap, int* __restrict__ status) {
  __shared__ uint32_t sh_warp[WARPS];
  const uint64_t w0 = static_cast<uint64_t>(blockIdx.x) * WIRE_CHUNK_WORDS + threadIdx.x * WIRE_WORDS_PER_THREAD;
  uint32_t v[WIRE_WORDS_PER_THREAD];
  uint32_t c = 0;
#pragma unroll
  for (uint32_t q = 0; q < WIRE_WORDS_PER_THREAD; ++q) {
    v[q] = (w0 + q < n_words) ? words[w0 + q] : 0u;
    c += __popc(v[q]);
  }
  uint32_t total;
  uint64_t pos = static_cast<uint64_t>(chunk_off[blockIdx.x]) + block_excl_scan(c, sh_warp, total);
#pragma unroll
  for (uint32_t q = 0; q < WIRE_WORDS_PER_THREAD; ++q) {
    for (uint32_t bits = v[q]; bits; bits &= bits - 1) {
      const uint32_t i = static_cast<uint32_t>((w0 + q) << 5) + (__ffs(bits) - 1);
      if (pos < cap) idx[pos] = i; else atomicMin(status, STATUS_CAPACITY);
      ++pos;
    }
  }
}

}  // namespace iwp

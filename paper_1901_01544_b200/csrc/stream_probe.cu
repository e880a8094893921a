// Stand-alone probe of what the streaming pass of the pruning step can reach on a GPU: it moves the same
// bytes per element pair as step (a) (read residual and gradient, write residual: a += g) with the
// streaming kernel's SHAPE but none of its logic, in several variants, and prints the achieved bandwidth.
// It answers three design questions with measurements instead of guesses:
//   1. the ceiling for this access pattern (one warp walks one 4096-element tile in 512-element segments,
//      the next segment's 128-bit loads in flight, 7 warps x 3 CTAs per SM);
//   2. how much shared memory per CTA costs (shared memory is carved out of the L1, which tracks the loads
//      in flight);
//   3. whether staging the tiles through TMA bulk copies (cp.async.bulk + mbarrier ring) beats plain loads.
// Every wait on an mbarrier is bounded: after SPIN_LIMIT polls the CTA sets an error flag, waits for its own
// copies and returns.  No cluster multicast is used.
//
//   build:  python paper_1901_01544_b200/build.py --probe     run:  paper_1901_01544_b200/stream_probe [tiles]
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>

namespace {

constexpr int TILE = 4096;  // floats per tile (16 KB), as in the library
constexpr uint32_t SPIN_LIMIT = 1u << 22;

// ---- plain 128-bit streaming loads: one warp per tile, ROUNDS x 128 elements per lane and segment ----------
template <int ROUNDS, int WARPS_PER_CTA, int MIN_CTAS>
__global__ void __launch_bounds__(WARPS_PER_CTA * 32, MIN_CTAS)
    k_walk(const float* __restrict__ g, float* __restrict__ a, uint64_t n_tiles, int touch_pad) {
  extern __shared__ unsigned char pad[];  // only there to take shared memory away from the L1
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint64_t t = static_cast<uint64_t>(blockIdx.x) * WARPS_PER_CTA + warp;
  if (t >= n_tiles) return;
  if (touch_pad) pad[threadIdx.x] = 0;
  constexpr int SEG = ROUNDS * 128;
  const float4* g4 = reinterpret_cast<const float4*>(g + t * TILE) + lane;
  float4* a4 = reinterpret_cast<float4*>(a + t * TILE) + lane;
  float4 x[ROUNDS], y[ROUNDS], xn[ROUNDS], yn[ROUNDS];
#pragma unroll
  for (int s = 0; s < ROUNDS; ++s) {
    xn[s] = __ldcs(a4 + s * 32);
    yn[s] = __ldcs(g4 + s * 32);
  }
#pragma unroll 1
  for (int it = 0; it < TILE / SEG; ++it) {
#pragma unroll
    for (int s = 0; s < ROUNDS; ++s) {
      x[s] = xn[s];
      y[s] = yn[s];
    }
    if (it + 1 < TILE / SEG) {
#pragma unroll
      for (int s = 0; s < ROUNDS; ++s) {
        xn[s] = __ldcs(a4 + (it + 1) * SEG / 4 + s * 32);
        yn[s] = __ldcs(g4 + (it + 1) * SEG / 4 + s * 32);
      }
    }
#pragma unroll
    for (int s = 0; s < ROUNDS; ++s) {
      x[s].x += y[s].x;
      x[s].y += y[s].y;
      x[s].z += y[s].z;
      x[s].w += y[s].w;
      __stcs(a4 + it * SEG / 4 + s * 32, x[s]);
    }
  }
}

// ---- TMA 1-D bulk copies staged through a shared-memory ring, persistent CTAs ------------------------------
constexpr int TMA_THREADS = 256;
constexpr int STAGES = 3;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}

// Tile i of a CTA uses stage i % STAGES.  Thread 0 issues the bulk loads (completion on the stage's mbarrier)
// and the bulk store of each finished tile; a stage is refilled only after the store that read it is done.
__global__ void __launch_bounds__(TMA_THREADS) k_tma(const float* __restrict__ g, float* __restrict__ a, uint64_t n_tiles, int* err) {
  extern __shared__ __align__(128) unsigned char smem[];
  float* sa = reinterpret_cast<float*>(smem);  // [STAGES][TILE]
  float* sg = sa + STAGES * TILE;              // [STAGES][TILE]
  __shared__ __align__(8) unsigned long long bars[STAGES];
  __shared__ int failed;
  if (threadIdx.x == 0) {
    failed = 0;
    for (int s = 0; s < STAGES; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint64_t first = blockIdx.x, stride = gridDim.x;
  const uint64_t mine = first < n_tiles ? (n_tiles - first + stride - 1) / stride : 0;
  auto issue = [&](uint64_t i) {
    const int s = static_cast<int>(i % STAGES);
    const uint64_t t = first + i * stride;
    const uint32_t bar = smem_u32(&bars[s]);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2u * TILE * 4u) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(sa + s * TILE)),
                 "l"(a + t * TILE), "r"(TILE * 4u), "r"(bar)
                 : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(sg + s * TILE)),
                 "l"(g + t * TILE), "r"(TILE * 4u), "r"(bar)
                 : "memory");
  };
  if (threadIdx.x == 0)
    for (uint64_t i = 0; i < mine && i < STAGES - 1; ++i) issue(i);
  for (uint64_t i = 0; i < mine; ++i) {
    const int s = static_cast<int>(i % STAGES);
    if (threadIdx.x == 0 && i + STAGES - 1 < mine) {
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the stage's last store has read it
      issue(i + STAGES - 1);
    }
    if (!mbar_wait(smem_u32(&bars[s]), static_cast<uint32_t>((i / STAGES) & 1))) failed = 1;
    __syncthreads();
    if (failed) break;
    float4* xa = reinterpret_cast<float4*>(sa + s * TILE);
    const float4* xg = reinterpret_cast<const float4*>(sg + s * TILE);
#pragma unroll
    for (int q = 0; q < TILE / 4 / TMA_THREADS; ++q) {
      float4 x = xa[q * TMA_THREADS + threadIdx.x];
      const float4 y = xg[q * TMA_THREADS + threadIdx.x];
      x.x += y.x;
      x.y += y.y;
      x.z += y.z;
      x.w += y.w;
      xa[q * TMA_THREADS + threadIdx.x] = x;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
      const uint64_t t = first + i * stride;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(a + t * TILE), "r"(smem_u32(xa)), "r"(TILE * 4u)
                   : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
  }
  if (threadIdx.x == 0) {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (failed) atomicExch(err, 1);
  }
}

struct Bench {
  const float* g;
  float* a;
  uint64_t n_tiles;
  cudaEvent_t e0, e1;
  double gbs(float ms) const { return 3.0 * static_cast<double>(n_tiles) * TILE * 4 / ms / 1e6; }
};

template <typename K>
void run_walk(const Bench& b, const char* name, K kern, int warps, size_t smem) {
  cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  int occ = 0;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, warps * 32, smem);
  float best = 1e9f;
  for (int rep = 0; rep < 6; ++rep) {
    cudaEventRecord(b.e0);
    kern<<<static_cast<unsigned>((b.n_tiles + warps - 1) / warps), warps * 32, smem>>>(b.g, b.a, b.n_tiles, 0);
    cudaEventRecord(b.e1);
    cudaEventSynchronize(b.e1);
    float ms;
    cudaEventElapsedTime(&ms, b.e0, b.e1);
    if (rep && ms < best) best = ms;
  }
  std::printf("%-58s %d CTAs/SM = %2d warps  %.3f ms  %5.0f GB/s  %s\n", name, occ, occ * warps, best, b.gbs(best),
              cudaGetErrorString(cudaGetLastError()));
}

void run_tma(const Bench& b, const char* name, int ctas_per_sm, int sm_count, int* err) {
  const size_t dyn = 2 * STAGES * TILE * 4;
  cudaFuncSetAttribute(k_tma, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(dyn));
  float best = 1e9f;
  for (int rep = 0; rep < 6; ++rep) {
    cudaEventRecord(b.e0);
    k_tma<<<sm_count * ctas_per_sm, TMA_THREADS, dyn>>>(b.g, b.a, b.n_tiles, err);
    cudaEventRecord(b.e1);
    cudaEventSynchronize(b.e1);
    float ms;
    cudaEventElapsedTime(&ms, b.e0, b.e1);
    if (rep && ms < best) best = ms;
  }
  int h = 0;
  cudaMemcpy(&h, err, sizeof(int), cudaMemcpyDeviceToHost);
  std::printf("%-58s %d CTAs/SM             %.3f ms  %5.0f GB/s  %s%s\n", name, ctas_per_sm, best, b.gbs(best),
              cudaGetErrorString(cudaGetLastError()), h ? "  (a bounded wait gave up)" : "");
}

}  // namespace

int main(int argc, char** argv) {
  const uint64_t n_tiles = argc > 1 ? std::strtoull(argv[1], nullptr, 10) : 120000;  // 120000 tiles = 1.97 GB per array
  if (n_tiles < 1 || n_tiles > 400000) {
    std::fprintf(stderr, "tiles must be in 1..400000 (at most 6.6 GB per array)\n");
    return 2;
  }
  const uint64_t n = n_tiles * TILE;
  float *a = nullptr, *g = nullptr;
  int* err = nullptr;
  if (cudaMalloc(&a, n * 4) != cudaSuccess || cudaMalloc(&g, n * 4) != cudaSuccess || cudaMalloc(&err, sizeof(int)) != cudaSuccess) {
    std::fprintf(stderr, "allocation failed: %s\n", cudaGetErrorString(cudaGetLastError()));
    return 1;
  }
  cudaMemset(a, 0, n * 4);
  cudaMemset(g, 0, n * 4);
  cudaMemset(err, 0, sizeof(int));
  Bench b{g, a, n_tiles, nullptr, nullptr};
  cudaEventCreate(&b.e0);
  cudaEventCreate(&b.e1);
  int sm_count = 148;
  cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, 0);
  std::printf("a += g over 2 x %.2f GB (read 2, write 1), best of 5 timed launches each\n", n * 4 / 1e9);
  run_walk(b, "plain loads, 4 rounds, 7 warps, 16 KB smem (the library's shape)", k_walk<4, 7, 3>, 7, 16384);
  run_walk(b, "plain loads, 4 rounds, 7 warps, 26 KB smem", k_walk<4, 7, 3>, 7, 26624);
  run_walk(b, "plain loads, 4 rounds, 8 warps, 26 KB smem", k_walk<4, 8, 3>, 8, 26624);
  run_walk(b, "plain loads, 4 rounds, 8 warps, 26 KB smem, 4 CTAs wanted", k_walk<4, 8, 4>, 8, 26624);
  run_walk(b, "plain loads, 8 rounds, 8 warps, 26 KB smem", k_walk<8, 8, 3>, 8, 26624);
  run_walk(b, "plain loads, 4 rounds, 7 warps, 50 KB smem", k_walk<4, 7, 4>, 7, 51200);
  run_walk(b, "plain loads, 4 rounds, 7 warps, 70 KB smem", k_walk<4, 7, 3>, 7, 71680);
  run_tma(b, "TMA bulk copies, 3 stages x 32 KB", 1, sm_count, err);
  run_tma(b, "TMA bulk copies, 3 stages x 32 KB", 2, sm_count, err);
  cudaFree(a);
  cudaFree(g);
  cudaFree(err);
  return 0;
}

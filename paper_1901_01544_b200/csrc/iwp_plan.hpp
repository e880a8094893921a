// Host-side planner: turns a layer-size list into the tables the kernels walk.
// Pure C++ (no CUDA): also used by iwp_plan_sizes(), which runs without a GPU.
//
// Every tensor is one selection unit (Algorithm 1 loops over layers j = 0..M).  Layers of at
// most SMALL_MAX elements take the one-CTA path (the whole (worker, layer) problem fits in
// shared memory); all others are cut into tiles and chunks:
//   tile   <= TILE consecutive elements of ONE layer, never crossing a multiple of TILE of the
//          flat element space, so that a tile is at most TILE/4 aligned 128-bit slots;
//   chunk  <= CHUNK_TILES consecutive tiles of one layer: the unit of work of the select kernels (8 .. 128
//          tiles, by the size of the job: see chunk_tiles_for).
#pragma once
#include <cmath>
#include <cstddef>
#include <cstdint>
#include <vector>

namespace iwp {

constexpr uint32_t TILE = 4096;
constexpr uint32_t CHUNK_TILES = 128;      // largest chunk
constexpr uint32_t CHUNK_TILES_MIN = 8;
constexpr uint32_t SMALL_MAX = 16384;
constexpr uint32_t NBINS = 2048;
constexpr int32_t MAX_WORKERS = 65535;  // workers index the y dimension of several grids
// single-read path: capacity of a (tile, worker) candidate slot and the sample that sets the guess
constexpr uint32_t CAND_CAP = 512;
constexpr uint32_t SAMPLE_MAX = 16384;
constexpr uint32_t GUESS_NONE = 0xffffffffu;  // no importance pattern reaches this value
constexpr uint32_t SEG_ELEMS = 512;           // elements a warp handles per iteration of the streaming pass
constexpr uint32_t SEGS_PER_TILE = TILE / SEG_ELEMS;
// single-read path, one-launch select: a (layer, worker) pair of at most this many tiles is selected and listed
// by one CTA from its candidate slots; larger layers take the multi-launch chain
constexpr uint32_t PAIR_MAX_TILES = 640;
constexpr uint32_t REF_NONE = 0xffffffffu;    // list entry has no side values: gather from the residuals, zero them
constexpr uint32_t REF_LAZY = 0xfffffffeu;    // the same, but leave the zeroing to the next streaming pass

struct LayerDesc {
  uint32_t off;         // flat offset of the first element
  uint32_t n;           // elements
  uint32_t k;           // keep count
  uint32_t koff;        // offset of the layer's segment inside a worker's list
  int32_t large_index;  // index among tiled layers, -1 on the one-CTA path
  uint32_t first_tile;  // tiled layers: first tile / chunk and their counts
  uint32_t n_tiles;
  uint32_t first_chunk;
  uint32_t n_chunks;
  uint32_t sample;  // elements sampled for the threshold guess (multiple of 8), 0 = no speculation
  uint32_t rho;     // the guess is the rho-th largest sampled importance
};

struct Tile {
  uint32_t a;      // first element (flat)
  uint32_t len;    // 1..TILE
  uint32_t layer;  // owning layer
  uint32_t large_index;
};

struct Chunk {
  uint32_t a;           // first element (flat)
  uint32_t len;         // elements
  uint32_t layer;       // owning layer
  uint32_t first_tile;  // first tile of the chunk
  uint32_t n_tiles;
  uint32_t first_chunk_of_layer;
};

// Tiles per chunk for a job of total_tiles tiles and W workers.  A (chunk, worker) is one CTA of the select
// kernels, which are latency bound: a small job cut into 128-tile chunks would run them on a handful of SMs
// (one layer of 2^20 elements and four workers: 8 CTAs), while cutting a large job finer only multiplies the
// per-chunk histogram merges and suffix tables (measured slower).  At least about 256 CTAs per launch where
// the job has them, 8 to 128 tiles per chunk, a power of two.
inline uint32_t chunk_tiles_for(uint64_t total_tiles, int32_t W) {
  uint32_t ct = CHUNK_TILES_MIN;
  while (ct < CHUNK_TILES && static_cast<uint64_t>(ct) * 2 * 256 <= total_tiles * static_cast<uint64_t>(W)) ct *= 2;
  return ct;
}

inline int64_t keep_count(int64_t n, double ratio) {
  if (n < 1 || !(ratio >= 1.0) || !std::isfinite(ratio)) return 0;
  double q = std::ceil(static_cast<double>(n) / ratio);
  int64_t k = static_cast<int64_t>(q);
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
}

// Sample size s and rank rho for the threshold guess of a tiled layer.  With p = k/n the number of
// sampled elements above the true threshold is ~Binomial(s, p); taking the rho-th largest sample with
// rho = s p + 4.5 sqrt(s p (1-p)) + 2 puts the guess below the true threshold except with probability
// ~1e-5 (then the exact multi-pass select takes over for that pair).  Speculation is switched off when
// the expected candidate density rho/s would fill more than a third of a candidate slot.
inline void sample_plan(uint32_t n, uint32_t k, uint32_t* sample, uint32_t* rho) {
  *sample = 0;
  *rho = 0;
  if (k >= n) return;
  uint32_t s = (n / 16) & ~7u;
  if (s > SAMPLE_MAX) s = SAMPLE_MAX;
  if (s < 64) return;
  const double p = static_cast<double>(k) / static_cast<double>(n);
  const double mean = s * p;
  const double r = std::ceil(mean + 4.5 * std::sqrt(mean * (1.0 - p)) + 2.0);
  if (r * 24.0 > static_cast<double>(s)) return;
  *sample = s;
  *rho = static_cast<uint32_t>(r);
}

inline uint64_t mix64(uint64_t z) {
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

inline int32_t leader_at(uint64_t seed, uint64_t t, int32_t W) {
  if (W < 1) return -1;
  const uint64_t z = mix64(seed + (t + 1) * 0x9E3779B97F4A7C15ull);
  return static_cast<int32_t>(((z >> 32) * static_cast<uint64_t>(W)) >> 32);
}

// The chosen node of layer l at step t when every layer draws its own (option "per_layer_leaders").
#if defined(__CUDACC__)
__host__ __device__
#endif
inline int32_t layer_leader_at(uint64_t seed, uint64_t t, uint64_t l, int32_t W) {
  uint64_t z = seed + (t + 1) * 0x9E3779B97F4A7C15ull + (l + 1) * 0xA0761D6478BD642Full;
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return static_cast<int32_t>(((z >> 32) * static_cast<uint64_t>(W)) >> 32);
}

// Section 3.3, random gradient selection: the 24-bit uniform draw of element i at step t.
#if defined(__CUDACC__)
__host__ __device__
#endif
inline uint32_t draw24(uint64_t seed, uint64_t t, uint64_t i) {
  uint64_t z = seed + (t + 1) * 0x9E3779B97F4A7C15ull + (i + 1) * 0xC2B2AE3D27D4EB4Full;
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return static_cast<uint32_t>(z >> 40);
}

// Chosen nodes r_1..r_n of step t: n distinct workers drawn without replacement; r_1 = leader_at().
constexpr int MAX_LEADERS = 8;
struct LeaderSet {
  int32_t n;
  int32_t r[MAX_LEADERS];
};

inline LeaderSet leaders_at(uint64_t seed, uint64_t t, int32_t W, int32_t n) {
  LeaderSet ls{};
  ls.n = n;
  std::vector<int32_t> remaining(static_cast<size_t>(W));
  for (int32_t w = 0; w < W; ++w) remaining[static_cast<size_t>(w)] = w;
  for (int32_t j = 0; j < n; ++j) {
    const uint64_t z = mix64(seed + (t + 1) * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(j) * 0xD1B54A32D192ED03ull);
    const uint64_t u = ((z >> 32) * static_cast<uint64_t>(W - j)) >> 32;
    ls.r[j] = remaining[u];
    remaining.erase(remaining.begin() + static_cast<std::ptrdiff_t>(u));
  }
  return ls;
}

struct Plan {
  std::vector<LayerDesc> layers;
  std::vector<Tile> tiles;
  std::vector<Chunk> chunks;
  std::vector<uint32_t> small_layers;  // layer ids on the one-CTA path
  std::vector<uint32_t> large_layers;  // layer ids on the tiled path
  // tiled layers by how the single-read path selects: one CTA per (layer, worker) pair, or the chain of
  // histogram / digit / compaction launches over chunks
  std::vector<uint32_t> pair_layers;   // layer ids
  std::vector<uint32_t> chain_large;   // indices among the tiled layers
  std::vector<uint32_t> chain_chunks;  // chunk ids
  uint64_t N = 0, K = 0;
  uint32_t max_small_n = 0;
  int32_t W = 0;
  bool valid = false;
};

// small_max: layers of at most this many elements take the one-CTA path (0: every layer is tiled, no
// threshold sampling - the plan of the absolute-threshold mode, which also uses smaller chunks because
// its select kernels walk one worker only and need the parallelism).  chunk_tiles = 0: by layer size.
inline Plan make_plan(const int64_t* sizes, int32_t n_layers, int32_t W, double ratio, float eps,
                      uint32_t small_max = SMALL_MAX, uint32_t chunk_tiles_fixed = 0) {
  Plan p;
  if (!sizes || n_layers < 1 || W < 1 || W > MAX_WORKERS || !(ratio >= 1.0) || !std::isfinite(ratio) ||
      !(eps > 0.f) || !std::isfinite(eps))
    return p;
  uint64_t N = 0;
  for (int32_t l = 0; l < n_layers; ++l) {
    if (sizes[l] < 1) return p;
    N += static_cast<uint64_t>(sizes[l]);
    if (N >= (1ull << 32)) return p;
  }
  p.W = W;
  uint64_t total_tiles = 0;  // of the tiled layers (an upper estimate: ragged layer ends add a tile here and there)
  for (int32_t l = 0; l < n_layers; ++l)
    if (static_cast<uint64_t>(sizes[l]) > small_max) total_tiles += (static_cast<uint64_t>(sizes[l]) + TILE - 1) / TILE;
  const uint32_t chunk_tiles = chunk_tiles_fixed ? chunk_tiles_fixed : chunk_tiles_for(total_tiles, W);
  uint64_t off = 0, koff = 0;
  for (int32_t l = 0; l < n_layers; ++l) {
    LayerDesc d{};
    d.off = static_cast<uint32_t>(off);
    d.n = static_cast<uint32_t>(sizes[l]);
    d.k = static_cast<uint32_t>(keep_count(sizes[l], ratio));
    d.koff = static_cast<uint32_t>(koff);
    d.large_index = -1;
    if (d.n <= small_max) {
      p.small_layers.push_back(static_cast<uint32_t>(l));
      if (d.n > p.max_small_n) p.max_small_n = d.n;
    } else {
      d.large_index = static_cast<int32_t>(p.large_layers.size());
      p.large_layers.push_back(static_cast<uint32_t>(l));
      d.first_tile = static_cast<uint32_t>(p.tiles.size());
      d.first_chunk = static_cast<uint32_t>(p.chunks.size());
      uint64_t a = off;
      const uint64_t end = off + d.n;
      while (a < end) {
        uint64_t b = (a / TILE + 1) * TILE;  // next multiple of TILE
        if (b > end) b = end;
        Tile t{static_cast<uint32_t>(a), static_cast<uint32_t>(b - a), static_cast<uint32_t>(l),
               static_cast<uint32_t>(d.large_index)};
        p.tiles.push_back(t);
        a = b;
      }
      d.n_tiles = static_cast<uint32_t>(p.tiles.size()) - d.first_tile;
      for (uint32_t t0 = 0; t0 < d.n_tiles; t0 += chunk_tiles) {
        const uint32_t nt = (d.n_tiles - t0 < chunk_tiles) ? d.n_tiles - t0 : chunk_tiles;
        Chunk c{};
        c.first_tile = d.first_tile + t0;
        c.n_tiles = nt;
        c.a = p.tiles[c.first_tile].a;
        const Tile& last = p.tiles[c.first_tile + nt - 1];
        c.len = last.a + last.len - c.a;
        c.layer = static_cast<uint32_t>(l);
        c.first_chunk_of_layer = d.first_chunk;
        p.chunks.push_back(c);
      }
      d.n_chunks = static_cast<uint32_t>(p.chunks.size()) - d.first_chunk;
      if (small_max != 0) sample_plan(d.n, d.k, &d.sample, &d.rho);
      if (d.sample != 0 && d.n_tiles <= PAIR_MAX_TILES) {
        p.pair_layers.push_back(static_cast<uint32_t>(l));
      } else {
        p.chain_large.push_back(static_cast<uint32_t>(d.large_index));
        for (uint32_t q = 0; q < d.n_chunks; ++q) p.chain_chunks.push_back(d.first_chunk + q);
      }
    }
    p.layers.push_back(d);
    off += d.n;
    koff += d.k;
  }
  p.N = off;
  p.K = koff;
  p.valid = true;
  return p;
}

}  // namespace iwp

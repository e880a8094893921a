// C ABI of the importance-weighted pruning step (see include/iwp.h): argument checks,
// the host planner, device memory owned by a context, and the launch sequence of a step.
//
// The sm_100a kernels live in the headers included below, by step of the path (Algorithm 1 of the paper):
//   iwp_device.cuh     shared device helpers (importance arithmetic, vector loads, scans, radix select)
//   iwp_sample.cuh     threshold guess of the single-read path from a sample of every (layer, worker) pair
//   iwp_stream.cuh     (a)+(b): accumulate, single-read streaming pass (importance, candidates, side values)
//   iwp_select.cuh     (c)+(d): exact radix select, ordered compaction, one-CTA path of small layers
//   iwp_reduce.cuh     (e)-(g): reduction at the index set, zero mask, sharded phases, mask accessor
//   iwp_threshold.cuh  absolute-threshold mode, random selection, layer-wise threshold
//   iwp_wire.cuh       index list <-> one-bit-per-element mask (the two wire formats of the sharded step)
// Nothing here is a dense contraction, so there are no tensor-core instructions: every kernel is bound by
// HBM traffic (or, for the small ones, by launch latency).  The residual add, the eps guard and the division
// use the explicit round-to-nearest intrinsics, so results do not depend on compiler contraction or fast-math
// flags, and denormals are kept.
#include "../../include/iwp.h"

#include <cuda_runtime.h>

#include <cmath>
#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "iwp_device.cuh"
#include "iwp_plan.hpp"
#include "iwp_reduce.cuh"
#include "iwp_sample.cuh"
#include "iwp_select.cuh"
#include "iwp_stream.cuh"
#include "iwp_threshold.cuh"
#include "iwp_wire.cuh"

using namespace iwp;

// Warps per CTA of the select kernels of one chain: histogram + digit kernels, compaction kernel.
struct ChainWidth {
  int hist, write;
};

struct iwp_ctx {
  Plan plan;
  float eps = 0.f;
  float momentum = 1.0f;  // Eq. 3: factor on the locally kept residual before the new gradient is added
  double ratio = 1.0;
  uint64_t seed = 0;
  int64_t t = 0;
  int32_t leader = -1;
  int64_t leader_override = -1;
  bool force_scalar = false;
  bool speculate = true;
  // option: layers of at most PAIR_MAX_TILES tiles are selected by one cluster launch (k_select_pair) instead of
  // the chain; -1 = decided by the size of the job at create (see below), 0 = never, 1 = always
  int pair_select = -1;
  bool pair_select_auto = false;
  bool select_only = false;  // iwp_shard_select(): a step stops before the reduction
  bool leader_only_select = false;  // option: only the chosen node selects; the other workers' lists are not produced
  cudaStream_t stream = nullptr;
  cudaStream_t side = nullptr;       // the one-CTA path of small layers runs here, beside the tiled path
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_fork2 = nullptr, ev_join2 = nullptr;
  // Overlapped schedule of the single-read path: the leader's select runs on side_a under the other
  // workers' streaming pass; the other workers' selects run on side_a (next step's leader) and side_b
  // (everybody else) beside the reduction and the head of the NEXT step, which waits for them just
  // before it overwrites what they read.
  int overlap = 1;  // 0 off, 1 on (the default is chosen by size at create)
  cudaStream_t side_a = nullptr, side_b = nullptr;
  cudaEvent_t ev_lead = nullptr, ev_lead_done = nullptr, ev_others = nullptr, ev_a2 = nullptr, ev_b = nullptr;
  bool pending_a2 = false, pending_b = false;  // deferred selects of the last step not yet joined
  // The three select chains of the overlapped schedule.  Histogram and digit kernels with four warps per CTA (64
  // registers a thread) fit into the registers the streaming pass leaves free on an SM, so they take no CTA slot
  // from it, but take longer; the chain of the next step's chosen node is waited for by that step's first launch
  // and keeps eight warps there and runs its compaction with sixteen warps per CTA (half the latency again); the other compactions keep eight
  // (with four they take twice as long and the next step waits).  Measured, ms per step on the AlexNet shape
  // W=8 / the ResNet-50 shape: eight warps everywhere 1.294 / 0.700; this choice 1.288 / 0.668; four everywhere in
  // the histogram kernels 1.306 / 0.673; sixteen in every compaction 1.292 / 0.673.
  ChainWidth cw_lead{4, 8}, cw_next{8, 16}, cw_rest{4, 8};
  int32_t predicted_next = -1;                 // the worker whose select pending_a2 covers
  int32_t last_only = -1;                      // the last step selected for this worker alone (-1: for every worker)
  float* saved_w = nullptr;                    // [N] weights kept for deferred selects that fall back (k_save_weights)
  int device = 0;
  int64_t launches = 0;
  uint64_t device_bytes = 0;
  uint32_t n_pairs = 0;  // (tiled layer, worker) pairs
  // device memory
  float* acc = nullptr;
  LayerDesc* d_layers = nullptr;
  Tile* d_tiles = nullptr;
  Chunk* d_chunks = nullptr;
  uint32_t* d_small_ids = nullptr;
  uint32_t* d_large_ids = nullptr;
  uint32_t* d_pair_ids = nullptr;      // layers the single-read path selects with one CTA per (layer, worker) pair
  uint32_t* d_chain_large = nullptr;   // the other tiled layers (indices among the tiled layers) ...
  uint32_t* d_chain_chunks = nullptr;  // ... and their chunks
  uint2* d_state = nullptr;
  uint32_t* d_hist = nullptr;
  int32_t* d_layer_leader = nullptr;  // [layer] chosen node of each layer (option "per_layer_leaders")
  uint32_t* d_reach = nullptr;    // [pair] candidates reaching the guess as the first histogram pass saw them (count check)
  uint2* d_chunk_cnt = nullptr;
  PairInfo* d_info = nullptr;     // threshold guess and candidate totals per pair, two copies used in turn
  PairInfo* info_cur = nullptr;   // the copy the last step used
  uint2* d_guess = nullptr;       // read-only (guess, pre-test multiplier) per pair for the streaming pass
  float* side_val = nullptr;      // every worker's value at the leader's slot positions, laid out like cand_val
  uint32_t* sel_slot = nullptr;   // [K] slot position of each entry of the leader's list, or REF_NONE
  uint2* lead_lane = nullptr;     // [segment][32] the leader's staged mask | count << 16, lane prefix
  uint32_t* lead_tot = nullptr;   // [segment] the leader's per-round totals
  uint32_t* chunk_sfx = nullptr;  // [W][chunk][1024] suffix sums of each chunk's last-pass histogram
  // absolute-threshold mode (Algorithm 1 as printed)
  bool threshold_mode = false;
  uint64_t list_cap = 0;          // capacity of the single index list
  bool thr_set = false;
  int32_t n_leaders = 1;          // chosen nodes whose masks are OR-ed
  LeaderSet last_chosen{};        // ratio mode: the chosen nodes of the last step
  bool per_layer_leaders = false; // ratio mode: every layer draws its own chosen node
  bool last_per_layer = false;    // the last step did so
  bool random_select = false;     // Section 3.3: P(update) = importance / threshold below the threshold
  uint32_t* d_thr = nullptr;      // [layer] fp32 patterns of the thresholds
  bool layerwise = false;         // Section 3.4: thresholds from each chosen node's per-layer statistics (Eq. 4)
  double lw_alpha = 0.0, lw_beta = 0.0, lw_c = 0.0;
  int32_t lw_chosen = 0;          // chosen nodes of the last layer-wise step
  uint32_t* d_thr_lw = nullptr;   // [chosen node][layer] fp32 patterns of the derived thresholds
  unsigned long long* d_bins = nullptr;  // [chosen node][layer][3][256] exact moment sums in the making
  uint32_t* d_tcnt = nullptr;     // [chunk] selected elements of the chunk
  uint32_t* d_toff = nullptr;     // [chunk] list offset of the chunk
  uint32_t* d_list_len = nullptr; // length of the last step's index list
  uint32_t* d_wire_cnt = nullptr; // [chunk of 32 Ki elements] set bits of a mask being expanded, then their offsets
  uint32_t* d_wire_off = nullptr;
  uint32_t* d_wire_len = nullptr; // length of the last expanded list
  uint32_t* zmask = nullptr;      // residuals sent in the last step and not yet zeroed (lazy step (g))
  uint64_t zmask_words = 0;
  bool zero_pending = false;      // zmask may hold marks
  uint32_t* cand_key = nullptr;   // candidate slots [tile][worker][CAND_CAP]
  float* cand_val = nullptr;
  uint16_t* cand_idx = nullptr;
  uint32_t* cand_cnt = nullptr;   // [tile][worker]
  bool info_clean = true;         // d_info holds "no guess" everywhere
  uint32_t max_sample = 0;
  uint32_t spec_pairs = 0;
  uint32_t* sel_idx = nullptr;
  float* sel_val = nullptr;
  int* d_status = nullptr;
  // optional per-stage CUDA-event timing (option "time_stages")
  int time_stages = 0;  // 0 off, 1 every stage boundary, 2 only around the dominant streaming stage
  std::vector<cudaEvent_t> stage_events;  // N_STAGES + 1 events per timed step
  std::vector<cudaEvent_t> event_pool;    // events made ahead of the timed steps (option "reserve_timed_steps")
  // staging for iwp_step_host
  float* stg_grads = nullptr;
  float* stg_weights = nullptr;
  float* stg_update = nullptr;
  // double-buffered staging of iwp_step_host_async: set k & 1 serves call k
  struct HostPipe {
    float* grads[2] = {nullptr, nullptr};
    float* weights[2] = {nullptr, nullptr};
    float* update[2] = {nullptr, nullptr};
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t in_ready[2] = {nullptr, nullptr};   // the set's inputs have arrived
    cudaEvent_t step_done[2] = {nullptr, nullptr};  // the step that used the set is through
    cudaEvent_t out_done[2] = {nullptr, nullptr};   // the set's update has reached the host
    int64_t calls = 0;
  } pipe_host;
};

namespace {

constexpr int WRITE_WARPS = 8;  // warps per CTA of the select kernels in the serial schedule

// stages of a step, in launch order; an event is recorded at every boundary when timing is on
enum Stage { ST_SMALL = 0, ST_SAMPLE, ST_ACCUMULATE, ST_SELECT, ST_COMPACT, ST_GATHER, N_STAGES };
const char* const kStageKeys[N_STAGES] = {"time_small_ns", "time_sample_ns", "time_accumulate_ns", "time_select_ns", "time_compact_ns",
                                          "time_gather_ns"};

// Called at every stage boundary of a step, in order; `boundary` = index of the stage that begins.
void stage_mark_at(iwp_ctx* c, int boundary) {
  if (!c->time_stages) return;
  cudaEvent_t e = nullptr;
  // the dominant stage: the streaming pass of the ratio mode, the fused all-worker pass of the threshold mode
  const int dominant = c->threshold_mode ? ST_GATHER : ST_ACCUMULATE;
  const bool wanted = c->time_stages == 1 || boundary == dominant || boundary == dominant + 1;
  if (wanted) {
    if (!c->event_pool.empty()) {  // made ahead of time: nothing but the record happens inside a timed step
      e = c->event_pool.back();
      c->event_pool.pop_back();
    } else if (cudaEventCreate(&e) != cudaSuccess) {
      cudaGetLastError();
      e = nullptr;
    }
    if (e) cudaEventRecord(e, c->stream);
  }
  c->stage_events.push_back(e);  // a null entry keeps the slots of a step aligned
}

void stage_clear(iwp_ctx* c) {
  for (cudaEvent_t e : c->stage_events)
    if (e) cudaEventDestroy(e);
  c->stage_events.clear();
  for (cudaEvent_t e : c->event_pool) cudaEventDestroy(e);
  c->event_pool.clear();
}

struct Sizes {
  uint64_t acc, layers, tiles, chunks, small_ids, large_ids, state, hist, reach, chunk_cnt, sel_idx, sel_val, status;
  uint64_t info, cand_key, cand_val, cand_idx, cand_cnt, guess, side_val, sel_slot, lead_lane, lead_tot, zmask, chunk_sfx;
  uint64_t saved_w;
  uint64_t total() const {
    return acc + layers + tiles + chunks + small_ids + large_ids + state + hist + reach + chunk_cnt + sel_idx + sel_val +
           status + info + cand_key + cand_val + cand_idx + cand_cnt + guess + side_val + sel_slot + lead_lane +
           lead_tot + zmask + chunk_sfx + saved_w;
  }
};

uint64_t at_least(uint64_t b) { return b ? b : 16; }

Sizes sizes_of(const Plan& p, bool threshold_mode = false, uint64_t list_cap = 0) {
  Sizes s;
  const uint64_t W = static_cast<uint64_t>(p.W);
  // the threshold mode selects on one worker only and needs none of the per-pair select scratch
  const uint64_t pairs = threshold_mode ? 0 : W * p.large_layers.size();
  s.acc = W * p.N * sizeof(float);
  s.layers = p.layers.size() * sizeof(LayerDesc);
  s.tiles = at_least(p.tiles.size() * sizeof(Tile));
  s.chunks = at_least(p.chunks.size() * sizeof(Chunk));
  s.small_ids = at_least(p.small_layers.size() * sizeof(uint32_t));
  s.large_ids = at_least(p.large_layers.size() * sizeof(uint32_t));
  s.state = at_least(pairs * sizeof(uint2));
  s.hist = at_least(pairs * NBINS * sizeof(uint32_t));
  s.reach = at_least(pairs * sizeof(uint32_t));
  s.chunk_cnt = at_least((threshold_mode ? 0 : W) * p.chunks.size() * sizeof(uint2));
  s.sel_idx = threshold_mode ? at_least(list_cap * sizeof(uint32_t)) : W * p.K * sizeof(uint32_t);
  s.sel_val = threshold_mode ? at_least(list_cap * sizeof(float)) : W * p.K * sizeof(float);
  s.status = sizeof(int);
  bool any_spec = false;
  for (uint32_t l : p.large_layers) any_spec = any_spec || p.layers[l].sample != 0;
  const uint64_t slots = any_spec ? W * p.tiles.size() : 0;
  s.info = at_least(2 * pairs * sizeof(PairInfo));
  s.cand_key = at_least(slots * CAND_CAP * sizeof(uint32_t));
  s.cand_val = at_least(slots * CAND_CAP * sizeof(float));
  s.cand_idx = at_least(slots * CAND_CAP * sizeof(uint16_t));
  s.cand_cnt = at_least(slots * sizeof(uint32_t));
  const uint64_t segs = any_spec ? p.tiles.size() * SEGS_PER_TILE : 0;
  s.guess = at_least(pairs * sizeof(uint2));
  s.side_val = at_least(slots * CAND_CAP * sizeof(float));
  s.sel_slot = at_least((threshold_mode ? 0 : p.K) * sizeof(uint32_t));
  s.lead_lane = at_least(segs * 32 * sizeof(uint2));
  s.lead_tot = at_least(segs * sizeof(uint32_t));
  s.zmask = ((p.N >> 9) + 2) * 16 * sizeof(uint32_t);  // 32 sixteen-bit fields per 512 elements
  s.chunk_sfx = at_least((threshold_mode ? 0 : W) * p.chunks.size() * pass_bins(N_PASSES - 1) * sizeof(uint32_t));
  s.saved_w = at_least((any_spec && !threshold_mode && W > 1) ? p.N * sizeof(float) : 0);
  return s;
}

template <typename T>
int dev_alloc(T** p, uint64_t bytes) {
  void* q = nullptr;
  const cudaError_t e = cudaMalloc(&q, bytes);
  if (e == cudaErrorMemoryAllocation) {
    cudaGetLastError();
    return IWP_ERR_OOM;
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  *p = static_cast<T*>(q);
  return IWP_OK;
}

void free_all(iwp_ctx* c) {
  if (c->side) {
    cudaStreamSynchronize(c->side);
    cudaStreamDestroy(c->side);
  }
  for (cudaStream_t* q : {&c->side_a, &c->side_b}) {
    if (*q) {
      cudaStreamSynchronize(*q);
      cudaStreamDestroy(*q);
    }
  }
  for (cudaEvent_t e : {c->ev_lead, c->ev_lead_done, c->ev_others, c->ev_a2, c->ev_b})
    if (e) cudaEventDestroy(e);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->ev_fork2) cudaEventDestroy(c->ev_fork2);
  if (c->ev_join2) cudaEventDestroy(c->ev_join2);
  cudaFree(c->acc);
  cudaFree(c->d_layers);
  cudaFree(c->d_tiles);
  cudaFree(c->d_chunks);
  cudaFree(c->d_small_ids);
  cudaFree(c->d_large_ids);
  cudaFree(c->d_pair_ids);
  cudaFree(c->d_chain_large);
  cudaFree(c->d_chain_chunks);
  cudaFree(c->d_state);
  cudaFree(c->d_hist);
  cudaFree(c->d_reach);
  cudaFree(c->d_layer_leader);
  cudaFree(c->d_chunk_cnt);
  cudaFree(c->d_info);
  cudaFree(c->cand_key);
  cudaFree(c->cand_val);
  cudaFree(c->cand_idx);
  cudaFree(c->cand_cnt);
  cudaFree(c->d_guess);
  cudaFree(c->side_val);
  cudaFree(c->sel_slot);
  cudaFree(c->lead_lane);
  cudaFree(c->lead_tot);
  cudaFree(c->zmask);
  cudaFree(c->d_thr);
  cudaFree(c->d_thr_lw);
  cudaFree(c->d_bins);
  cudaFree(c->d_tcnt);
  cudaFree(c->d_toff);
  cudaFree(c->d_list_len);
  cudaFree(c->d_wire_cnt);
  cudaFree(c->d_wire_off);
  cudaFree(c->d_wire_len);
  cudaFree(c->chunk_sfx);
  cudaFree(c->saved_w);
  cudaFree(c->sel_idx);
  cudaFree(c->sel_val);
  cudaFree(c->d_status);
  cudaFree(c->stg_grads);
  cudaFree(c->stg_weights);
  cudaFree(c->stg_update);
  {
    iwp_ctx::HostPipe& hp = c->pipe_host;
    for (cudaStream_t* q : {&hp.h2d, &hp.d2h})
      if (*q) {
        cudaStreamSynchronize(*q);
        cudaStreamDestroy(*q);
      }
    for (int k = 0; k < 2; ++k) {
      cudaFree(hp.grads[k]);
      cudaFree(hp.weights[k]);
      cudaFree(hp.update[k]);
      for (cudaEvent_t e : {hp.in_ready[k], hp.step_done[k], hp.out_done[k]})
        if (e) cudaEventDestroy(e);
    }
  }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#define IWP_LAUNCH_CHECK(c)                         \
  do {                                              \
    (c)->launches += 1;                             \
    if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA; \
  } while (0)

// Makes the main stream wait for the selects a previous step left running on the side streams.
int join_deferred(iwp_ctx* c) {
  bool ok = true;
  if (c->pending_a2) ok = cudaStreamWaitEvent(c->stream, c->ev_a2, 0) == cudaSuccess && ok;
  if (c->pending_b) ok = cudaStreamWaitEvent(c->stream, c->ev_b, 0) == cudaSuccess && ok;
  c->pending_a2 = c->pending_b = false;
  if (!ok) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

// Brings the residuals themselves up to date when the last step left its zeroing to the next
// streaming pass (see k_sum_scatter) and somebody else is about to look at them.
int flush_pending_zero(iwp_ctx* c) {
  if (const int rc = join_deferred(c)) return rc;  // a deferred select may still be reading the residuals
  if (!c->zero_pending) return IWP_OK;
  const unsigned blocks = static_cast<unsigned>((c->zmask_words + THREADS - 1) / THREADS);
  k_flush_zmask<<<blocks, THREADS, 0, c->stream>>>(c->zmask, c->acc, c->zmask_words, c->plan.N, c->plan.W);
  c->launches += 1;
  if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  c->zero_pending = false;
  return IWP_OK;
}

// Which tiled layers the chain of histogram / digit / compaction launches covers in a step.
struct ChainScope {
  const uint32_t* chunk_ids;  // nullptr: every chunk
  const uint32_t* large_sel;  // nullptr: every tiled layer
  unsigned n_chunks, n_large;
  bool pairs;                 // the layers left out are selected by k_select_pair
};

// With speculation the layers of at most PAIR_MAX_TILES tiles are selected and listed by one CTA per pair.
ChainScope chain_scope(const iwp_ctx* c, bool spec) {
  const Plan& p = c->plan;
  const bool on = c->pair_select < 0 ? c->pair_select_auto : c->pair_select == 1;
  if (spec && on && !p.pair_layers.empty())
    return ChainScope{c->d_chain_chunks, c->d_chain_large, static_cast<unsigned>(p.chain_chunks.size()),
                      static_cast<unsigned>(p.chain_large.size()), true};
  return ChainScope{nullptr, nullptr, static_cast<unsigned>(p.chunks.size()), static_cast<unsigned>(p.large_layers.size()), false};
}

template <bool VEC>
int launch_pair_select(iwp_ctx* c, const float* weights, cudaStream_t st, WorkerSel ws, int32_t leader,
                       const int32_t* lead_tab) {
  const Plan& p = c->plan;
  const unsigned n_sel = static_cast<unsigned>(sel_count(ws, p.W));
  if (n_sel == 0 || p.pair_layers.empty()) return IWP_OK;
  k_select_pair<VEC><<<dim3(static_cast<unsigned>(p.pair_layers.size()) * PAIR_CLUSTER, n_sel), THREADS,
                       PAIR_KEYS_SMEM * sizeof(uint32_t), st>>>(
      c->acc, weights, c->d_tiles, c->d_layers, c->d_pair_ids, c->info_cur, c->cand_key, c->cand_val, c->cand_idx,
      c->cand_cnt, c->d_state, c->sel_idx, c->sel_val, c->sel_slot, c->d_status, c->eps, p.N, p.K, p.W, leader, ws, lead_tab);
  IWP_LAUNCH_CHECK(c);
  return IWP_OK;
}

template <bool VEC, int HW, int WW>
int select_and_write_w(iwp_ctx* c, const float* weights, cudaStream_t st, WorkerSel ws, int32_t leader) {
  const Plan& p = c->plan;
  const int W = p.W;
  const unsigned n_chunks = static_cast<unsigned>(p.chunks.size());
  const unsigned n_sel = static_cast<unsigned>(sel_count(ws, W));
  if (n_sel == 0) return IWP_OK;
  const ChainScope sc = chain_scope(c, true);
  if (sc.pairs) {
    const int rc = launch_pair_select<VEC>(c, weights, st, ws, leader, nullptr);
    if (rc != IWP_OK) return rc;
  }
  if (sc.n_chunks == 0) return IWP_OK;
  dim3 cgrid(sc.n_chunks, n_sel), pgrid(sc.n_large, n_sel);
  uint32_t* sfx = c->chunk_sfx;
  for (int pass = 0; pass < N_PASSES; ++pass) {
    k_hist<VEC, HW><<<cgrid, HW * 32, 0, st>>>(c->acc, weights, c->d_chunks, c->d_layers, c->info_cur, c->cand_key,
                                               c->cand_cnt, c->d_state, c->d_hist, sfx, c->d_chunk_cnt, c->d_reach, c->eps,
                                               p.N, W, pass, n_chunks, ws, sc.chunk_ids);
    IWP_LAUNCH_CHECK(c);
    k_find_digit<HW><<<pgrid, HW * 32, 0, st>>>(c->d_state, c->d_hist, c->d_layers, c->d_large_ids, c->info_cur, c->d_reach,
                                                c->d_status, W, pass, ws, sc.large_sel);
    IWP_LAUNCH_CHECK(c);
  }
  k_write<VEC, WW><<<cgrid, WW * 32, 0, st>>>(
      c->acc, weights, c->d_chunks, c->d_tiles, c->d_layers, c->info_cur, c->cand_key, c->cand_val, c->cand_idx, c->cand_cnt,
      c->d_state, c->d_chunk_cnt, c->sel_idx, c->sel_val, c->sel_slot, sfx, c->d_status, c->eps, p.N, p.K, W, n_chunks, leader,
      ws, nullptr, sc.chunk_ids);
  IWP_LAUNCH_CHECK(c);
  return IWP_OK;
}

// Exact select and ordered compaction of the workers `ws` covers, on stream `st` (single-read path): one
// launch for the layers selected per pair, the chain (three histogram passes with their digit decisions, then
// the compaction) for the others.
template <bool VEC>
int select_and_write(iwp_ctx* c, const float* weights, cudaStream_t st, WorkerSel ws, int32_t leader, ChainWidth cw) {
  if (cw.hist == 16) {
    return cw.write == 16 ? select_and_write_w<VEC, 16, 16>(c, weights, st, ws, leader)
                          : select_and_write_w<VEC, 16, 8>(c, weights, st, ws, leader);
  }
  if (cw.hist == 4) {
    return cw.write == 16 ? select_and_write_w<VEC, 4, 16>(c, weights, st, ws, leader)
                          : select_and_write_w<VEC, 4, 8>(c, weights, st, ws, leader);
  }
  return cw.write == 16 ? select_and_write_w<VEC, 8, 16>(c, weights, st, ws, leader)
                        : select_and_write_w<VEC, 8, 8>(c, weights, st, ws, leader);
}

int32_t leader_of_step(const iwp_ctx* c, int64_t t) {
  return c->leader_override >= 0 ? static_cast<int32_t>(c->leader_override)
                                 : leader_at(c->seed, static_cast<uint64_t>(t), c->plan.W);
}

template <bool VEC>
int run_step(iwp_ctx* c, const float* grads, const float* weights, float* update, int32_t leader) {
  const Plan& p = c->plan;
  const int W = p.W;
  const uint64_t N = p.N, K = p.K;
  cudaStream_t s = c->stream;
  auto cuda_ok = [](cudaError_t e) {
    if (e == cudaSuccess) return true;
    cudaGetLastError();
    return false;
  };
  const bool tiled = !p.large_layers.empty();
  const bool spec = tiled && c->speculate && c->spec_pairs > 0;
  // several chosen nodes (their lists are OR-ed) unless the leader is forced; r_1 is `leader` either way
  LeaderSet ls{};
  if (c->n_leaders > 1 && c->leader_override < 0) {
    ls = leaders_at(c->seed, static_cast<uint64_t>(c->t), W, c->n_leaders);
  } else {
    ls.n = 1;
    ls.r[0] = leader;
  }
  c->last_chosen = ls;
  const bool per_layer = c->per_layer_leaders && c->leader_override < 0 && ls.n == 1 && !c->select_only;
  c->last_per_layer = per_layer;
  // only the chosen node's list is consumed by the step: with the option on, nobody else selects
  const bool only = c->leader_only_select && W > 1 && ls.n == 1 && !per_layer && !c->select_only;
  const int only_w = only ? leader : -1;
  c->last_only = only_w;
  // the overlapped schedule (not while every stage boundary is being timed)
  const bool pipe = spec && W > 1 && ls.n == 1 && !per_layer && !c->select_only && c->overlap == 1 && c->time_stages != 1 &&
                    c->side_a != nullptr && c->side_b != nullptr;
  if (!pipe) {
    const int rc = join_deferred(c);
    if (rc != IWP_OK) return rc;
  }
  if (!spec) {  // the multi-pass path reads the residuals as they are (before the small layers' kernel adds to them)
    const int rc = flush_pending_zero(c);
    if (rc != IWP_OK) return rc;
  }
  // one chosen node per layer: the table the kernels read it from (single-read path; the multi-pass path draws
  // the nodes inside its reduction kernel)
  const int32_t* lead_tab = nullptr;
  if (per_layer && spec) {
    const unsigned nl = static_cast<unsigned>(p.layers.size());
    k_layer_leaders<<<(nl + THREADS - 1) / THREADS, THREADS, 0, s>>>(c->d_layer_leader, nl, c->seed,
                                                                    static_cast<uint64_t>(c->t), W);
    IWP_LAUNCH_CHECK(c);
    lead_tab = c->d_layer_leader;
  }
  stage_mark_at(c, 0);
  // Small layers touch nothing the tiled path touches until the final reduction, so when both kinds
  // exist their one-CTA kernel runs on a side stream, forked here and joined before the reduction.
  const bool fork_small = !p.small_layers.empty() && tiled && c->side != nullptr;
  if (!p.small_layers.empty()) {
    const size_t dyn = static_cast<size_t>(p.max_small_n) * sizeof(uint32_t);
    dim3 grid(static_cast<unsigned>(p.small_layers.size()), static_cast<unsigned>(W));
    cudaStream_t ss = s;
    if (fork_small) {
      if (!cuda_ok(cudaEventRecord(c->ev_fork, s)) || !cuda_ok(cudaStreamWaitEvent(c->side, c->ev_fork, 0)))
        return IWP_ERR_CUDA;
      ss = c->side;
    }
    k_small<<<grid, THREADS, dyn, ss>>>(grads, weights, c->acc, update, c->d_layers, c->d_small_ids, c->sel_idx,
                                        c->sel_val, c->sel_slot, c->d_status, c->eps, N, K, leader, only_w, c->momentum,
                                        lead_tab);
    IWP_LAUNCH_CHECK(c);
    if (fork_small && !cuda_ok(cudaEventRecord(c->ev_join, c->side))) return IWP_ERR_CUDA;
  }
  stage_mark_at(c, 1);
  // The per-pair records alternate between two copies, so that a select still running for the last
  // step keeps reading its own while this step's sampling writes the other.
  c->info_cur = c->d_info + static_cast<size_t>(c->t & 1) * c->n_pairs;
  if (tiled && !spec && !c->info_clean) {  // speculation was switched off: forget the old guesses
    if (!cuda_ok(cudaMemsetAsync(c->d_info, 0xff, 2 * static_cast<size_t>(c->n_pairs) * sizeof(PairInfo), s)))
      return IWP_ERR_CUDA;
    c->launches += 1;
    c->info_clean = true;
  }
  if (spec) {
    const size_t dyn = static_cast<size_t>(c->max_sample) * sizeof(uint32_t);
    k_sample<<<c->n_pairs, SAMPLE_THREADS, dyn, s>>>(grads, weights, c->acc, c->d_layers, c->d_large_ids, c->info_cur,
                                                     c->d_guess, c->zmask, c->eps, N, W, static_cast<uint32_t>(c->t),
                                                     only_w, c->momentum);
    IWP_LAUNCH_CHECK(c);
    c->info_clean = false;
  }
  const unsigned n_tiles = static_cast<unsigned>(p.tiles.size());
  const unsigned gblocks = static_cast<unsigned>((K + THREADS - 1) / THREADS);
  if (!pipe) stage_mark_at(c, 2);
  if (pipe) {
    // This step's leader was covered by side_a's deferred select if the last step foresaw it; any
    // other worker may still be in side_b's.
    if (c->pending_a2 && !cuda_ok(cudaStreamWaitEvent(s, c->ev_a2, 0))) return IWP_ERR_CUDA;
    c->pending_a2 = false;
    if (c->pending_b && leader != c->predicted_next) {
      if (!cuda_ok(cudaStreamWaitEvent(s, c->ev_b, 0))) return IWP_ERR_CUDA;
      c->pending_b = false;
    }
    stage_mark_at(c, 2);  // after the wait: the streaming stage is timed from where its first kernel may start
    k_stream<VEC, true><<<(n_tiles + WARPS - 1) / WARPS, THREADS, 0, s>>>(
        grads, weights, c->acc, update, c->d_tiles, c->info_cur, c->d_guess, c->cand_key, c->cand_val, c->cand_idx,
        c->cand_cnt, c->side_val, c->lead_lane, c->lead_tot, c->zmask, c->eps, N, W, leader, n_tiles, 1, c->momentum, c->d_status, lead_tab);
    IWP_LAUNCH_CHECK(c);
    // the leader's select and list, under the other workers' streaming pass
    if (!cuda_ok(cudaEventRecord(c->ev_lead, s)) || !cuda_ok(cudaStreamWaitEvent(c->side_a, c->ev_lead, 0)))
      return IWP_ERR_CUDA;
    int rc = select_and_write<VEC>(c, weights, c->side_a, WorkerSel{WorkerSel::ONLY, leader, -1}, leader, c->cw_lead);
    if (rc != IWP_OK) return rc;
    if (!cuda_ok(cudaEventRecord(c->ev_lead_done, c->side_a))) return IWP_ERR_CUDA;
    if (c->pending_b && !cuda_ok(cudaStreamWaitEvent(s, c->ev_b, 0))) return IWP_ERR_CUDA;
    c->pending_b = false;
    const int wpc = (W - 1 < WARPS) ? W - 1 : WARPS;  // warps (= workers) per CTA
    const int groups = (W - 1 + wpc - 1) / wpc;
    k_stream<VEC, false><<<n_tiles * static_cast<unsigned>(groups), wpc * 32, 0, s>>>(
        grads, weights, c->acc, update, c->d_tiles, c->info_cur, c->d_guess, c->cand_key, c->cand_val, c->cand_idx,
        c->cand_cnt, c->side_val, c->lead_lane, c->lead_tot, c->zmask, c->eps, N, W, leader, n_tiles, groups,
        c->momentum, c->d_status, lead_tab);
    IWP_LAUNCH_CHECK(c);
    if (c->zero_pending) {  // every marked residual has now been overwritten: forget the marks
      if (!cuda_ok(cudaMemsetAsync(c->zmask, 0, c->zmask_words * sizeof(uint32_t), s))) return IWP_ERR_CUDA;
      c->launches += 1;
      c->zero_pending = false;
    }
    stage_mark_at(c, 3);
    stage_mark_at(c, 4);
    stage_mark_at(c, 5);
    const int32_t next = leader_of_step(c, c->t + 1);
    if (!only) {
    // The other workers' selects outlive the step: they read the library's copy of the weights
    // (filled only where a pair fell back), the next step's leader first (its streaming pass comes first).
    k_save_weights<<<static_cast<unsigned>(p.chunks.size()), THREADS, 0, s>>>(weights, c->saved_w, c->d_chunks, c->d_layers,
                                                                            c->info_cur, W, leader);
    IWP_LAUNCH_CHECK(c);
    if (!cuda_ok(cudaEventRecord(c->ev_others, s))) return IWP_ERR_CUDA;
    if (next != leader) {
      if (!cuda_ok(cudaStreamWaitEvent(c->side_a, c->ev_others, 0))) return IWP_ERR_CUDA;
      rc = select_and_write<VEC>(c, c->saved_w, c->side_a, WorkerSel{WorkerSel::ONLY, next, -1}, leader, c->cw_next);
      if (rc != IWP_OK) return rc;
      if (!cuda_ok(cudaEventRecord(c->ev_a2, c->side_a))) return IWP_ERR_CUDA;
      c->pending_a2 = true;
    }
    const WorkerSel rest{WorkerSel::EXCEPT, leader, next};
    if (sel_count(rest, W) > 0) {
      if (!cuda_ok(cudaStreamWaitEvent(c->side_b, c->ev_others, 0))) return IWP_ERR_CUDA;
      rc = select_and_write<VEC>(c, c->saved_w, c->side_b, rest, leader, c->cw_rest);
      if (rc != IWP_OK) return rc;
      if (!cuda_ok(cudaEventRecord(c->ev_b, c->side_b))) return IWP_ERR_CUDA;
      c->pending_b = true;
    }
    }
    c->predicted_next = next;
    // the reduction needs the leader's list and the small layers
    if (!cuda_ok(cudaStreamWaitEvent(s, c->ev_lead_done, 0))) return IWP_ERR_CUDA;
    if (fork_small && !cuda_ok(cudaStreamWaitEvent(s, c->ev_join, 0))) return IWP_ERR_CUDA;
    k_sum_scatter<<<gblocks, THREADS, 0, s>>>(c->sel_idx + static_cast<uint64_t>(leader) * K, c->sel_slot, c->side_val,
                                              c->cand_val, c->acc, update, c->zmask, N, K, W, leader,
                                              static_cast<uint64_t>(p.tiles.size()) * W, c->d_status, nullptr, 0u, nullptr, 0);
    IWP_LAUNCH_CHECK(c);
    c->zero_pending = true;
    stage_mark_at(c, 6);
    return IWP_OK;
  }
  if (tiled) {
    if (spec) {
      // the leader's worker first (records where its candidates sit), then everybody else
      k_stream<VEC, true><<<(n_tiles + WARPS - 1) / WARPS, THREADS, 0, s>>>(
          grads, weights, c->acc, update, c->d_tiles, c->info_cur, c->d_guess, c->cand_key, c->cand_val, c->cand_idx,
          c->cand_cnt, c->side_val, c->lead_lane, c->lead_tot, c->zmask, c->eps, N, W, leader, n_tiles, 1,
          c->momentum, c->d_status, lead_tab);
      if (W > 1) {
        IWP_LAUNCH_CHECK(c);
        const int wpc = (W - 1 < WARPS) ? W - 1 : WARPS;  // warps (= workers) per CTA
        const int groups = (W - 1 + wpc - 1) / wpc;
        k_stream<VEC, false><<<n_tiles * static_cast<unsigned>(groups), wpc * 32, 0, s>>>(
            grads, weights, c->acc, update, c->d_tiles, c->info_cur, c->d_guess, c->cand_key, c->cand_val, c->cand_idx,
            c->cand_cnt, c->side_val, c->lead_lane, c->lead_tot, c->zmask, c->eps, N, W, leader, n_tiles, groups,
            c->momentum, c->d_status, lead_tab);
      }
      if (c->zero_pending) {  // every marked residual has now been overwritten: forget the marks
        IWP_LAUNCH_CHECK(c);
        if (!cuda_ok(cudaMemsetAsync(c->zmask, 0, c->zmask_words * sizeof(uint32_t), s))) return IWP_ERR_CUDA;
        c->zero_pending = false;
      }
    } else {
      k_accumulate<VEC><<<n_tiles, THREADS, 0, s>>>(grads, c->acc, update, c->d_tiles, N, W, c->momentum);
    }
    IWP_LAUNCH_CHECK(c);
  }
  stage_mark_at(c, 3);
  bool join_others = false;  // the other workers' lists are still being written on the side stream
  if (tiled) {
    const unsigned n_chunks = static_cast<unsigned>(p.chunks.size());
    const WorkerSel all = only ? WorkerSel{WorkerSel::ONLY, leader, -1} : WorkerSel{WorkerSel::ALL, 0, -1};
    const unsigned n_sel = static_cast<unsigned>(sel_count(all, W));
    const ChainScope sc = chain_scope(c, spec);
    if (sc.pairs) {  // select and list in one launch for the layers small enough for one CTA per pair
      const int rc = launch_pair_select<VEC>(c, weights, s, all, leader, lead_tab);
      if (rc != IWP_OK) return rc;
    }
    dim3 cgrid(sc.n_chunks, n_sel), pgrid(sc.n_large, n_sel);
    for (int pass = 0; pass < N_PASSES && sc.n_chunks > 0; ++pass) {
      k_hist<VEC, WRITE_WARPS><<<cgrid, WRITE_WARPS * 32, 0, s>>>(c->acc, weights, c->d_chunks, c->d_layers, c->info_cur, c->cand_key,
                                            c->cand_cnt, c->d_state, c->d_hist, c->chunk_sfx, c->d_chunk_cnt, c->d_reach,
                                            c->eps, N, W, pass, n_chunks, all, sc.chunk_ids);
      IWP_LAUNCH_CHECK(c);
      k_find_digit<WRITE_WARPS><<<pgrid, WRITE_WARPS * 32, 0, s>>>(c->d_state, c->d_hist, c->d_layers, c->d_large_ids, c->info_cur, c->d_reach,
                                             c->d_status, W, pass, all, sc.large_sel);
      IWP_LAUNCH_CHECK(c);
    }
    stage_mark_at(c, 4);
    // The reduction needs the leader's list only: write that one here and the other workers' lists on
    // the side stream, beside the reduction; they are joined at the end of the step.
    // (a union needs every chosen node's list here, a sharded step every list)
    const bool split = spec && W > 1 && ls.n == 1 && !per_layer && !c->select_only && !only && c->side != nullptr;
    auto write = [&](cudaStream_t st, WorkerSel ws) {
      if (sc.n_chunks == 0) return;
      dim3 grid(sc.n_chunks, static_cast<unsigned>(sel_count(ws, W)));
      k_write<VEC, WRITE_WARPS><<<grid, WRITE_WARPS * 32, 0, st>>>(c->acc, weights, c->d_chunks, c->d_tiles, c->d_layers, c->info_cur,
                                             c->cand_key, c->cand_val, c->cand_idx, c->cand_cnt, c->d_state,
                                             c->d_chunk_cnt, c->sel_idx, c->sel_val, c->sel_slot, c->chunk_sfx,
                                             c->d_status, c->eps, N, K, W, n_chunks, leader, ws, lead_tab, sc.chunk_ids);
    };
    if (split) {
      if (!cuda_ok(cudaEventRecord(c->ev_fork2, s)) || !cuda_ok(cudaStreamWaitEvent(c->side, c->ev_fork2, 0)))
        return IWP_ERR_CUDA;
      write(c->side, WorkerSel{WorkerSel::EXCEPT, leader, -1});
      IWP_LAUNCH_CHECK(c);
      if (!cuda_ok(cudaEventRecord(c->ev_join2, c->side))) return IWP_ERR_CUDA;
      write(s, WorkerSel{WorkerSel::ONLY, leader, -1});
      IWP_LAUNCH_CHECK(c);
      join_others = true;
    } else {
      write(s, all);
      IWP_LAUNCH_CHECK(c);
    }
  } else {
    stage_mark_at(c, 4);
  }
  stage_mark_at(c, 5);
  if (fork_small && !cuda_ok(cudaStreamWaitEvent(s, c->ev_join, 0))) return IWP_ERR_CUDA;
  if (c->select_only) {  // the reduction is the caller's (iwp_shard_gather / iwp_shard_apply)
    stage_mark_at(c, 6);
    return IWP_OK;
  }
  if (per_layer && spec) {
    // every worker's value at its layer's chosen node's candidate positions came out of the streaming pass
    k_sum_scatter<<<gblocks, THREADS, 0, s>>>(c->sel_idx, c->sel_slot, c->side_val, c->cand_val, c->acc, update, c->zmask,
                                              N, K, W, leader, static_cast<uint64_t>(p.tiles.size()) * W, c->d_status,
                                              c->d_layers, static_cast<uint32_t>(p.layers.size()), lead_tab, 0);
    c->zero_pending = true;
  } else if (per_layer) {
    k_layer_leader_sum_scatter<<<gblocks, THREADS, 0, s>>>(c->sel_idx, c->d_layers, static_cast<uint32_t>(p.layers.size()),
                                                           c->acc, update, nullptr, N, K, W, c->seed,
                                                           static_cast<uint64_t>(c->t));
  } else if (ls.n > 1) {
    // union of the chosen nodes' lists: the zero mask is all clear here (applied and cleared by the streaming
    // pass, or flushed at the start of a multi-pass step) and serves to give every element one owner
    // r_1 played the chosen node's part in the streaming pass, so its list is reduced from the side values; only
    // the elements that r_2 .. r_n add to the union are gathered from the residuals
    const int first_node = spec ? 1 : 0;
    if (spec) {
      k_sum_scatter<<<gblocks, THREADS, 0, s>>>(c->sel_idx + static_cast<uint64_t>(leader) * K, c->sel_slot, c->side_val,
                                                c->cand_val, c->acc, update, c->zmask, N, K, W, leader,
                                                static_cast<uint64_t>(p.tiles.size()) * W, c->d_status, nullptr, 0u, nullptr, 1);
      IWP_LAUNCH_CHECK(c);
    }
    const uint64_t entries = static_cast<uint64_t>(ls.n - first_node) * K;
    k_union_sum_scatter<<<static_cast<unsigned>((entries + THREADS - 1) / THREADS), THREADS, 0, s>>>(
        c->sel_idx, c->acc, update, c->zmask, N, K, W, ls, c->d_layers, static_cast<uint32_t>(p.layers.size()), first_node);
    c->zero_pending = true;  // the marks are cleared with the next step's
  } else if (spec) {
    k_sum_scatter<<<gblocks, THREADS, 0, s>>>(c->sel_idx + static_cast<uint64_t>(leader) * K, c->sel_slot, c->side_val,
                                              c->cand_val, c->acc, update, c->zmask, N, K, W, leader,
                                              static_cast<uint64_t>(p.tiles.size()) * W, c->d_status, nullptr, 0u, nullptr, 0);
    c->zero_pending = true;
  } else {
    k_gather_sum_scatter<<<gblocks, THREADS, 0, s>>>(c->sel_idx + static_cast<uint64_t>(leader) * K, c->acc, update,
                                                     N, K, W);
  }
  IWP_LAUNCH_CHECK(c);
  if (join_others && !cuda_ok(cudaStreamWaitEvent(s, c->ev_join2, 0))) return IWP_ERR_CUDA;
  stage_mark_at(c, 6);
  return IWP_OK;
}

}  // namespace

extern "C" {

const char* iwp_strerror(int status) {
  switch (status) {
    case IWP_OK: return "ok";
    case IWP_ERR_INVALID: return "invalid argument";
    case IWP_ERR_OOM: return "out of memory";
    case IWP_ERR_CUDA: return "CUDA runtime error";
    case IWP_ERR_INTERNAL: return "device-side count check failed";
    case IWP_ERR_TIMEOUT: return "device-side wait timed out";
    case IWP_ERR_CAPACITY: return "index list longer than its capacity";
    default: return "unknown status";
  }
}

int64_t iwp_keep_count(int64_t n, double ratio) { return keep_count(n, ratio); }

int32_t iwp_leader_at(uint64_t seed, uint64_t t, int32_t W) { return leader_at(seed, t, W); }

int32_t iwp_layer_leader_at(uint64_t seed, uint64_t t, int32_t layer, int32_t W) {
  if (W < 1 || layer < 0) return -1;
  return layer_leader_at(seed, t, static_cast<uint64_t>(layer), W);
}

int iwp_leaders_at(uint64_t seed, uint64_t t, int32_t W, int32_t n, int32_t* out) {
  if (!out || W < 1 || n < 1 || n > W || n > MAX_LEADERS) return IWP_ERR_INVALID;
  const LeaderSet ls = leaders_at(seed, t, W, n);
  for (int32_t j = 0; j < n; ++j) out[j] = ls.r[j];
  return IWP_OK;
}

int iwp_plan_sizes(const int64_t* layer_sizes, int32_t n_layers, int32_t W, double ratio, int64_t out[8]) {
  if (!out) return IWP_ERR_INVALID;
  const Plan p = make_plan(layer_sizes, n_layers, W, ratio, 1.0f);
  if (!p.valid) return IWP_ERR_INVALID;
  out[0] = static_cast<int64_t>(p.N);
  out[1] = static_cast<int64_t>(p.K);
  out[2] = static_cast<int64_t>(p.small_layers.size());
  out[3] = static_cast<int64_t>(p.large_layers.size());
  out[4] = static_cast<int64_t>(p.tiles.size());
  out[5] = static_cast<int64_t>(p.chunks.size());
  out[6] = static_cast<int64_t>(sizes_of(p).total());
  out[7] = (p.N % 4 == 0) ? 1 : 0;
  return IWP_OK;
}

}  // extern "C"

namespace {

constexpr uint32_t THRESHOLD_CHUNK_TILES = 8;  // 32 Ki elements per CTA of the threshold-mode passes over the chosen nodes

int create_common(iwp_ctx** out, const int64_t* layer_sizes, int32_t n_layers, int32_t W, double ratio, float eps,
                  uint64_t seed, bool threshold_mode, int64_t max_list) {
  if (!out) return IWP_ERR_INVALID;
  *out = nullptr;
  if (threshold_mode && max_list < 0) return IWP_ERR_INVALID;
  iwp_ctx* c = new (std::nothrow) iwp_ctx;
  if (!c) return IWP_ERR_OOM;
  try {
    c->plan = make_plan(layer_sizes, n_layers, W, ratio, eps, threshold_mode ? 0u : SMALL_MAX,
                        threshold_mode ? THRESHOLD_CHUNK_TILES : 0u);
  } catch (...) {
    delete c;
    return IWP_ERR_OOM;
  }
  if (!c->plan.valid) {
    delete c;
    return IWP_ERR_INVALID;
  }
  const Plan& p = c->plan;
  c->eps = eps;
  c->ratio = ratio;
  c->seed = seed;
  c->threshold_mode = threshold_mode;
  c->list_cap = threshold_mode ? ((max_list == 0 || static_cast<uint64_t>(max_list) > p.N) ? p.N : static_cast<uint64_t>(max_list)) : 0;
  c->n_pairs = static_cast<uint32_t>(p.large_layers.size()) * static_cast<uint32_t>(W);
  if (cudaGetDevice(&c->device) != cudaSuccess) {
    cudaGetLastError();
    delete c;
    return IWP_ERR_CUDA;
  }
  const Sizes sz = sizes_of(p, threshold_mode, c->list_cap);
  const uint64_t lw_thr_bytes = MAX_LEADERS * p.layers.size() * sizeof(uint32_t);
  const uint64_t lw_bin_bytes = MAX_LEADERS * p.layers.size() * 3 * LW_BINS * sizeof(unsigned long long);
  const uint64_t thr_bytes = threshold_mode
                                 ? (p.layers.size() + 2 * p.chunks.size() + 1) * sizeof(uint32_t) + lw_thr_bytes + lw_bin_bytes
                                 : 0;
  c->device_bytes = sz.total() + thr_bytes;
  int rc = IWP_OK;
  auto A = [&](auto** ptr, uint64_t bytes) {
    if (rc == IWP_OK) rc = dev_alloc(ptr, bytes);
  };
  A(&c->acc, sz.acc);
  A(&c->d_layers, sz.layers);
  A(&c->d_tiles, sz.tiles);
  A(&c->d_chunks, sz.chunks);
  A(&c->d_small_ids, sz.small_ids);
  A(&c->d_large_ids, sz.large_ids);
  A(&c->d_pair_ids, at_least(p.pair_layers.size() * sizeof(uint32_t)));
  A(&c->d_chain_large, at_least(p.chain_large.size() * sizeof(uint32_t)));
  A(&c->d_chain_chunks, at_least(p.chain_chunks.size() * sizeof(uint32_t)));
  A(&c->d_state, sz.state);
  A(&c->d_hist, sz.hist);
  A(&c->d_reach, sz.reach);
  A(&c->d_layer_leader, p.layers.size() * sizeof(int32_t));
  A(&c->d_chunk_cnt, sz.chunk_cnt);
  A(&c->d_info, sz.info);
  A(&c->cand_key, sz.cand_key);
  A(&c->cand_val, sz.cand_val);
  A(&c->cand_idx, sz.cand_idx);
  A(&c->cand_cnt, sz.cand_cnt);
  A(&c->d_guess, sz.guess);
  A(&c->side_val, sz.side_val);
  A(&c->sel_slot, sz.sel_slot);
  A(&c->lead_lane, sz.lead_lane);
  A(&c->lead_tot, sz.lead_tot);
  A(&c->zmask, sz.zmask);
  A(&c->chunk_sfx, sz.chunk_sfx);
  A(&c->saved_w, sz.saved_w);
  A(&c->sel_idx, sz.sel_idx);
  A(&c->sel_val, sz.sel_val);
  A(&c->d_status, sz.status);
  {
    const uint64_t wire_chunks = (((p.N + 31) >> 5) + WIRE_CHUNK_WORDS - 1) / WIRE_CHUNK_WORDS;
    A(&c->d_wire_cnt, wire_chunks * sizeof(uint32_t));
    A(&c->d_wire_off, wire_chunks * sizeof(uint32_t));
    A(&c->d_wire_len, sizeof(uint32_t));
    c->device_bytes += 2 * wire_chunks * sizeof(uint32_t) + sizeof(uint32_t);
  }
  if (threshold_mode) {
    A(&c->d_thr, p.layers.size() * sizeof(uint32_t));
    A(&c->d_tcnt, at_least(p.chunks.size() * sizeof(uint32_t)));
    A(&c->d_toff, at_least(p.chunks.size() * sizeof(uint32_t)));
    A(&c->d_list_len, sizeof(uint32_t));
    A(&c->d_thr_lw, lw_thr_bytes);
    A(&c->d_bins, lw_bin_bytes);
  }
  if (rc != IWP_OK) {
    free_all(c);
    delete c;
    return rc;
  }
  bool ok = true;
  if (threshold_mode) {
    ok = cudaMemset(c->d_list_len, 0, sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMemset(c->d_thr_lw, 0, lw_thr_bytes) == cudaSuccess;
    ok = ok && cudaMemset(c->d_bins, 0, lw_bin_bytes) == cudaSuccess;  // k_thr_finalize leaves them cleared
  }
  auto H2D = [&](void* dst, const void* src, size_t bytes) {
    if (bytes) ok = ok && cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice) == cudaSuccess;
  };
  H2D(c->d_layers, p.layers.data(), p.layers.size() * sizeof(LayerDesc));
  H2D(c->d_tiles, p.tiles.data(), p.tiles.size() * sizeof(Tile));
  H2D(c->d_chunks, p.chunks.data(), p.chunks.size() * sizeof(Chunk));
  H2D(c->d_small_ids, p.small_layers.data(), p.small_layers.size() * sizeof(uint32_t));
  H2D(c->d_large_ids, p.large_layers.data(), p.large_layers.size() * sizeof(uint32_t));
  H2D(c->d_pair_ids, p.pair_layers.data(), p.pair_layers.size() * sizeof(uint32_t));
  H2D(c->d_chain_large, p.chain_large.data(), p.chain_large.size() * sizeof(uint32_t));
  H2D(c->d_chain_chunks, p.chain_chunks.data(), p.chain_chunks.size() * sizeof(uint32_t));
  ok = ok && cudaMemset(c->acc, 0, sz.acc) == cudaSuccess;
  ok = ok && cudaMemset(c->d_state, 0, sz.state) == cudaSuccess;
  ok = ok && cudaMemset(c->d_hist, 0, sz.hist) == cudaSuccess;
  ok = ok && cudaMemset(c->d_reach, 0, sz.reach) == cudaSuccess;
  ok = ok && cudaMemset(c->d_chunk_cnt, 0, sz.chunk_cnt) == cudaSuccess;
  ok = ok && cudaMemset(c->sel_idx, 0, sz.sel_idx) == cudaSuccess;
  ok = ok && cudaMemset(c->sel_val, 0, sz.sel_val) == cudaSuccess;
  ok = ok && cudaMemset(c->d_status, 0, sz.status) == cudaSuccess;
  ok = ok && cudaMemset(c->d_info, 0xff, sz.info) == cudaSuccess;  // guess = none, overflow flag set
  ok = ok && cudaMemset(c->cand_cnt, 0, sz.cand_cnt) == cudaSuccess;
  ok = ok && cudaMemset(c->sel_slot, 0xff, sz.sel_slot) == cudaSuccess;
  ok = ok && cudaMemset(c->zmask, 0, sz.zmask) == cudaSuccess;
  c->zmask_words = sz.zmask / sizeof(uint32_t);
  for (uint32_t l : p.large_layers) {
    if (p.layers[l].sample > c->max_sample) c->max_sample = p.layers[l].sample;
    if (p.layers[l].sample) c->spec_pairs += static_cast<uint32_t>(W);
  }
  if (ok && c->max_sample) {
    ok = cudaFuncSetAttribute(k_sample, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(c->max_sample * sizeof(uint32_t))) == cudaSuccess;
  }
  if (ok && !p.pair_layers.empty()) {
    const int dyn = static_cast<int>(PAIR_KEYS_SMEM * sizeof(uint32_t));
    ok = cudaFuncSetAttribute(k_select_pair<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) == cudaSuccess;
    ok = ok && cudaFuncSetAttribute(k_select_pair<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) == cudaSuccess;
  }
  if (ok && p.max_small_n) {
    ok = cudaFuncSetAttribute(k_small, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              static_cast<int>(p.max_small_n * sizeof(uint32_t))) == cudaSuccess;
  }
  ok = ok && cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->ev_fork2, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&c->ev_join2, cudaEventDisableTiming) == cudaSuccess;
  if (ok && !threshold_mode) {
    int prio_lo = 0, prio_hi = 0;
    ok = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) == cudaSuccess;
    // The selects are short chains of small dependent kernels: at high priority their CTAs take the
    // next free slots of a streaming pass running beside them and the chains finish inside their windows.
    ok = ok && cudaStreamCreateWithPriority(&c->side_a, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
    ok = ok && cudaStreamCreateWithPriority(&c->side_b, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
    for (cudaEvent_t* e : {&c->ev_lead, &c->ev_lead_done, &c->ev_others, &c->ev_a2, &c->ev_b})
      ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
  }
  c->info_cur = c->d_info;
  // One cluster per (layer, worker) pair costs about 25 us whatever the pair's size (nine cluster barriers, three
  // histogram merges through distributed shared memory) and holds eight CTA slots meanwhile.  With a few pairs
  // that beats the seven dependent launches of the chain (one layer of 2^20 elements, four workers: select and
  // compaction 0.045 -> 0.027 ms); with hundreds of pairs the clusters queue up in waves while every launch of
  // the chain covers all pairs at once (161-tensor network shape, 368 pairs: 0.15 -> 0.30 ms).  So: by default
  // only for jobs of at most 64 pairs that have no layer left for the chain.
  c->pair_select_auto = !threshold_mode && p.chain_large.empty() && p.pair_layers.size() * static_cast<size_t>(W) <= 64;
  {  // the overlapped schedule costs extra launches: it pays once a step streams some hundred megabytes
    uint64_t tiled = 0;
    for (uint32_t l : p.large_layers) tiled += p.layers[l].n;
    c->overlap = (tiled * static_cast<uint64_t>(W) >= (1ull << 25)) ? 1 : 0;
  }
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    free_all(c);
    delete c;
    return IWP_ERR_CUDA;
  }
  *out = c;
  return IWP_OK;
}

// The threshold-mode step: accumulate the chosen nodes, count / scan / compact their masks into the
// index list and a bit per element, then one pass over all workers that accumulates the others, sums
// in worker order and zeroes at the set bits, and writes the dense update.
template <bool VEC>
int run_step_threshold(iwp_ctx* c, const float* grads, const float* weights, float* update, int32_t leader) {
  const Plan& p = c->plan;
  const int W = p.W;
  const uint64_t N = p.N;
  cudaStream_t s = c->stream;
  const unsigned n_tiles = static_cast<unsigned>(p.tiles.size());
  const unsigned n_chunks = static_cast<unsigned>(p.chunks.size());
  // several chosen nodes unless the leader is forced; r_1 is `leader` either way
  LeaderSet ls{};
  if (c->n_leaders > 1 && c->leader_override < 0) {
    ls = leaders_at(c->seed, static_cast<uint64_t>(c->t), W, c->n_leaders);
  } else {
    ls.n = 1;
    ls.r[0] = leader;
  }
  const uint32_t cap = static_cast<uint32_t>(c->list_cap);
  const RandomSelect rs{c->random_select ? 1 : 0, c->seed, static_cast<uint64_t>(c->t)};
  // (1) step (a) for the chosen nodes only; (2) their masks -> index list and a bit per element;
  // (3) one fused streaming pass over all workers: step (a) for the others, ordered sum, zeroing, update
  stage_mark_at(c, 0);
  stage_mark_at(c, 1);
  if (cudaMemsetAsync(c->zmask, 0, c->zmask_words * sizeof(uint32_t), s) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  c->launches += 1;
  stage_mark_at(c, 2);
  const uint32_t n_layers = static_cast<uint32_t>(p.layers.size());
  if (c->layerwise) {
    // Eq. 4 needs the accumulated residuals first: step (a) for the chosen nodes and their exact moments in one
    // pass, the thresholds, and only then the masks
    stage_mark_at(c, 3);
    k_thr_stats<VEC, true><<<dim3((n_chunks + STATS_GROUP - 1) / STATS_GROUP, static_cast<unsigned>(ls.n)), THREADS, 0, s>>>(
        c->acc, grads, weights, c->d_chunks, n_chunks, c->d_bins, c->eps, N, n_layers, c->momentum, ls);
    IWP_LAUNCH_CHECK(c);
    k_thr_finalize<<<dim3(n_layers, static_cast<unsigned>(ls.n)), THREADS, 0, s>>>(c->d_bins, c->d_layers, c->d_thr_lw, n_layers,
                                                                                c->lw_alpha, c->lw_beta, c->lw_c);
    IWP_LAUNCH_CHECK(c);
    c->lw_chosen = ls.n;
    k_thr_mask_count<VEC, false><<<n_chunks, THREADS, 0, s>>>(grads, c->acc, weights, c->d_chunks, c->d_thr_lw, n_layers,
                                                              c->zmask, c->d_tcnt, c->eps, N, c->momentum, ls, rs);
  } else {
    // fixed thresholds: step (a) for the chosen nodes, their masks and the chunk counts in one pass
    stage_mark_at(c, 3);
    k_thr_mask_count<VEC, true><<<n_chunks, THREADS, 0, s>>>(grads, c->acc, weights, c->d_chunks, c->d_thr, 0u, c->zmask,
                                                             c->d_tcnt, c->eps, N, c->momentum, ls, rs);
  }
  IWP_LAUNCH_CHECK(c);
  k_thr_scan<<<1, 1024, 0, s>>>(c->d_tcnt, c->d_toff, n_chunks, c->d_list_len);
  IWP_LAUNCH_CHECK(c);
  stage_mark_at(c, 4);
  k_thr_write<VEC><<<n_chunks, THREADS, 0, s>>>(c->acc + static_cast<uint64_t>(ls.r[0]) * N, c->d_chunks, c->d_toff, c->zmask,
                                                c->sel_idx, c->sel_val, cap, c->d_status);
  IWP_LAUNCH_CHECK(c);
  stage_mark_at(c, 5);
  k_thr_fused<VEC><<<n_tiles, THREADS, 0, s>>>(grads, c->acc, update, c->d_tiles, c->zmask, N, W, c->momentum, ls);
  IWP_LAUNCH_CHECK(c);
  stage_mark_at(c, 6);
  return IWP_OK;
}

}  // namespace

extern "C" {

int iwp_create(iwp_ctx** out, const int64_t* layer_sizes, int32_t n_layers, int32_t W, double ratio, float eps,
               uint64_t seed) {
  return create_common(out, layer_sizes, n_layers, W, ratio, eps, seed, false, 0);
}

int iwp_create_threshold(iwp_ctx** out, const int64_t* layer_sizes, int32_t n_layers, int32_t W, float eps,
                         uint64_t seed, int64_t max_list) {
  return create_common(out, layer_sizes, n_layers, W, 1.0, eps, seed, true, max_list);
}

int iwp_set_thresholds(iwp_ctx* c, const float* thr) {
  if (!c || !thr || !c->threshold_mode) return IWP_ERR_INVALID;
  std::vector<uint32_t> bits(c->plan.layers.size());
  for (size_t l = 0; l < bits.size(); ++l) {
    if (!(thr[l] >= 0.0f)) return IWP_ERR_INVALID;  // negative or NaN
    std::memcpy(&bits[l], &thr[l], sizeof(uint32_t));
    if (thr[l] == 0.0f) bits[l] = 0u;  // -0 is +0
  }
  // synchronous copy from a temporary: ordered after everything already enqueued on the stream
  if (cudaStreamSynchronize(c->stream) != cudaSuccess ||
      cudaMemcpy(c->d_thr, bits.data(), bits.size() * sizeof(uint32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  c->thr_set = true;
  return IWP_OK;
}

int iwp_set_layerwise(iwp_ctx* c, int32_t on, double alpha, double beta, double c_split) {
  if (!c || !c->threshold_mode || (on != 0 && on != 1)) return IWP_ERR_INVALID;
  if (on && (!std::isfinite(alpha) || !std::isfinite(beta) || !std::isfinite(c_split))) return IWP_ERR_INVALID;
  c->layerwise = on != 0;
  if (on) {
    c->lw_alpha = alpha;
    c->lw_beta = beta;
    c->lw_c = c_split;
  }
  return IWP_OK;
}

int iwp_get_layer_thresholds(iwp_ctx* c, float* dst, int32_t* n_chosen) {
  if (!c || !dst || !n_chosen || !c->threshold_mode || !c->layerwise) return IWP_ERR_INVALID;
  *n_chosen = c->lw_chosen;
  if (c->lw_chosen == 0) return IWP_OK;
  if (cudaMemcpyAsync(dst, c->d_thr_lw, static_cast<size_t>(c->lw_chosen) * c->plan.layers.size() * sizeof(uint32_t),
                      cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_get_list_length(iwp_ctx* c, int64_t* len) {
  if (!c || !len) return IWP_ERR_INVALID;
  if (!c->threshold_mode) {
    *len = static_cast<int64_t>(c->plan.K);
    return IWP_OK;
  }
  uint32_t v = 0;
  if (cudaMemcpyAsync(&v, c->d_list_len, sizeof(uint32_t), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaStreamSynchronize(c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  *len = static_cast<int64_t>(v);
  return IWP_OK;
}

int iwp_destroy(iwp_ctx* c) {
  if (!c) return IWP_OK;
  cudaStreamSynchronize(c->stream);
  stage_clear(c);
  free_all(c);
  cudaGetLastError();
  delete c;
  return IWP_OK;
}

int iwp_set_momentum(iwp_ctx* c, float m) {
  if (!c || !std::isfinite(m) || m < 0.f) return IWP_ERR_INVALID;
  c->momentum = m;
  return IWP_OK;
}

int iwp_set_stream(iwp_ctx* c, void* stream) {
  if (!c) return IWP_ERR_INVALID;
  // deferred selects were ordered against the old stream: let them finish before the switch
  if (c->pending_a2) cudaEventSynchronize(c->ev_a2);
  if (c->pending_b) cudaEventSynchronize(c->ev_b);
  c->pending_a2 = c->pending_b = false;
  cudaGetLastError();
  c->stream = static_cast<cudaStream_t>(stream);
  return IWP_OK;
}

int iwp_step(iwp_ctx* c, const float* grads, const float* weights, float* update) {
  if (!c || !grads || !weights || !update) return IWP_ERR_INVALID;
  const int32_t leader = c->leader_override >= 0 ? static_cast<int32_t>(c->leader_override)
                                                 : leader_at(c->seed, static_cast<uint64_t>(c->t), c->plan.W);
  const bool vec = !c->force_scalar && (c->plan.N % 4 == 0) && aligned16(grads) && aligned16(weights) &&
                   aligned16(update) && aligned16(c->acc);
  if (c->threshold_mode && !c->thr_set && !c->layerwise) return IWP_ERR_INVALID;  // no thresholds given yet
  const int rc = c->threshold_mode
                     ? (vec ? run_step_threshold<true>(c, grads, weights, update, leader)
                            : run_step_threshold<false>(c, grads, weights, update, leader))
                     : (vec ? run_step<true>(c, grads, weights, update, leader)
                            : run_step<false>(c, grads, weights, update, leader));
  if (rc != IWP_OK) return rc;
  c->leader = leader;
  c->t += 1;
  return IWP_OK;
}

int iwp_shard_select(iwp_ctx* c, const float* grads, const float* weights, float* update) {
  if (!c || !grads || !weights || !update || c->threshold_mode) return IWP_ERR_INVALID;
  const bool vec = !c->force_scalar && (c->plan.N % 4 == 0) && aligned16(grads) && aligned16(weights) &&
                   aligned16(update) && aligned16(c->acc);
  c->select_only = true;  // worker 0 plays the leader's part in the streaming pass; nothing is reduced
  const int rc = vec ? run_step<true>(c, grads, weights, update, 0) : run_step<false>(c, grads, weights, update, 0);
  c->select_only = false;
  if (rc != IWP_OK) return rc;
  c->leader = -1;
  return IWP_OK;
}

int iwp_shard_gather(iwp_ctx* c, const uint32_t* idx, int64_t n, float* vals) {
  if (!c || !idx || !vals || n < 0 || c->threshold_mode) return IWP_ERR_INVALID;
  if (const int rc = flush_pending_zero(c)) return rc;
  if (n == 0) return IWP_OK;
  const uint64_t total = static_cast<uint64_t>(n) * static_cast<uint64_t>(c->plan.W);
  const unsigned blocks = static_cast<unsigned>(std::min<uint64_t>((total + THREADS - 1) / THREADS, 148ull * 32));
  k_shard_gather<<<blocks, THREADS, 0, c->stream>>>(idx, c->acc, vals, c->plan.N, static_cast<uint64_t>(n), c->plan.W);
  IWP_LAUNCH_CHECK(c);
  return IWP_OK;
}

int iwp_shard_apply(iwp_ctx* c, const uint32_t* idx, int64_t n, const float* vals_all, int32_t W_total, float* update) {
  if (!c || !idx || !vals_all || !update || n < 0 || W_total < c->plan.W || c->threshold_mode) return IWP_ERR_INVALID;
  if (const int rc = flush_pending_zero(c)) return rc;
  if (n > 0) {
    const unsigned blocks = static_cast<unsigned>((static_cast<uint64_t>(n) + THREADS - 1) / THREADS);
    k_shard_apply<<<blocks, THREADS, 0, c->stream>>>(idx, vals_all, c->acc, update, c->zmask, c->d_layers,
                                                    static_cast<uint32_t>(c->plan.layers.size()), c->plan.N,
                                                    static_cast<uint64_t>(n), W_total, c->plan.W, c->d_status);
    IWP_LAUNCH_CHECK(c);
    c->zero_pending = true;  // the marks are the zeroing of the tiled layers' residuals
  }
  c->t += 1;
  return IWP_OK;
}

int iwp_step_host(iwp_ctx* c, const float* grads, const float* weights, float* update) {
  if (!c || !grads || !weights || !update) return IWP_ERR_INVALID;
  const uint64_t N = c->plan.N, W = static_cast<uint64_t>(c->plan.W);
  if (!c->stg_grads) {
    int rc = dev_alloc(&c->stg_grads, W * N * sizeof(float));
    if (rc == IWP_OK) rc = dev_alloc(&c->stg_weights, N * sizeof(float));
    if (rc == IWP_OK) rc = dev_alloc(&c->stg_update, N * sizeof(float));
    if (rc != IWP_OK) {
      cudaFree(c->stg_grads);
      cudaFree(c->stg_weights);
      cudaFree(c->stg_update);
      c->stg_grads = c->stg_weights = c->stg_update = nullptr;
      return rc;
    }
  }
  cudaStream_t s = c->stream;
  if (cudaMemcpyAsync(c->stg_grads, grads, W * N * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(c->stg_weights, weights, N * sizeof(float), cudaMemcpyHostToDevice, s) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  const int rc = iwp_step(c, c->stg_grads, c->stg_weights, c->stg_update);
  if (rc != IWP_OK) return rc;
  if (cudaMemcpyAsync(update, c->stg_update, N * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_step_host_async(iwp_ctx* c, const float* grads, const float* weights, float* update) {
  if (!c || !grads || !weights || !update) return IWP_ERR_INVALID;
  iwp_ctx::HostPipe& hp = c->pipe_host;
  const uint64_t N = c->plan.N, W = static_cast<uint64_t>(c->plan.W);
  if (!hp.h2d) {  // first call: two staging sets, a stream per copy direction, events
    int rc = IWP_OK;
    for (int k = 0; k < 2 && rc == IWP_OK; ++k) {
      rc = dev_alloc(&hp.grads[k], W * N * sizeof(float));
      if (rc == IWP_OK) rc = dev_alloc(&hp.weights[k], N * sizeof(float));
      if (rc == IWP_OK) rc = dev_alloc(&hp.update[k], N * sizeof(float));
    }
    bool ok = rc == IWP_OK;
    ok = ok && cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking) == cudaSuccess;
    for (int k = 0; k < 2; ++k)
      for (cudaEvent_t* e : {&hp.in_ready[k], &hp.step_done[k], &hp.out_done[k]})
        ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {  // free_all() releases whatever was made
      cudaGetLastError();
      return rc != IWP_OK ? rc : IWP_ERR_CUDA;
    }
  }
  const int k = static_cast<int>(hp.calls & 1);
  bool ok = true;
  if (hp.calls >= 2) {  // the set's last user: its step has read the inputs, its update has left
    ok = ok && cudaStreamWaitEvent(hp.h2d, hp.step_done[k], 0) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(c->stream, hp.out_done[k], 0) == cudaSuccess;
  }
  ok = ok && cudaMemcpyAsync(hp.grads[k], grads, W * N * sizeof(float), cudaMemcpyHostToDevice, hp.h2d) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(hp.weights[k], weights, N * sizeof(float), cudaMemcpyHostToDevice, hp.h2d) == cudaSuccess;
  ok = ok && cudaEventRecord(hp.in_ready[k], hp.h2d) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(c->stream, hp.in_ready[k], 0) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  const int rc = iwp_step(c, hp.grads[k], hp.weights[k], hp.update[k]);
  if (rc != IWP_OK) return rc;
  ok = cudaEventRecord(hp.step_done[k], c->stream) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(hp.d2h, hp.step_done[k], 0) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(update, hp.update[k], N * sizeof(float), cudaMemcpyDeviceToHost, hp.d2h) == cudaSuccess;
  ok = ok && cudaEventRecord(hp.out_done[k], hp.d2h) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  hp.calls += 1;
  return IWP_OK;
}

int iwp_host_wait(iwp_ctx* c) {
  if (!c) return IWP_ERR_INVALID;
  iwp_ctx::HostPipe& hp = c->pipe_host;
  if (!hp.d2h) return IWP_OK;
  if (cudaStreamSynchronize(hp.d2h) != cudaSuccess || cudaStreamSynchronize(c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_join(iwp_ctx* c) {
  if (!c) return IWP_ERR_INVALID;
  return join_deferred(c);
}

int iwp_sync_status(iwp_ctx* c) {
  if (!c) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  int st = 0;
  if (cudaMemcpyAsync(&st, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaStreamSynchronize(c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return st;
}

int iwp_get_layout(iwp_ctx* c, int64_t* off, int64_t* k) {
  if (!c) return IWP_ERR_INVALID;
  for (size_t l = 0; l < c->plan.layers.size(); ++l) {
    if (off) off[l] = c->plan.layers[l].off;
    if (k) k[l] = c->threshold_mode ? 0 : c->plan.layers[l].k;  // no fixed keep count under thresholds
  }
  return IWP_OK;
}

int iwp_get_sizes(iwp_ctx* c, int64_t out[4]) {
  if (!c || !out) return IWP_ERR_INVALID;
  out[0] = static_cast<int64_t>(c->plan.N);
  out[1] = static_cast<int64_t>(c->threshold_mode ? c->list_cap : c->plan.K);
  out[2] = static_cast<int64_t>(c->plan.layers.size());
  out[3] = c->plan.W;
  return IWP_OK;
}

int iwp_get_step(iwp_ctx* c, int64_t* t) {
  if (!c || !t) return IWP_ERR_INVALID;
  *t = c->t;
  return IWP_OK;
}

int iwp_set_step(iwp_ctx* c, int64_t t) {
  if (!c || t < 0) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  c->t = t;
  return IWP_OK;
}

int iwp_get_leader(iwp_ctx* c, int32_t* leader) {
  if (!c || !leader) return IWP_ERR_INVALID;
  *leader = c->leader;
  return IWP_OK;
}

int iwp_get_residual(iwp_ctx* c, int32_t w, float* dst) {
  if (!c || !dst || w < 0 || w >= c->plan.W) return IWP_ERR_INVALID;
  if (const int rc = flush_pending_zero(c)) return rc;
  const uint64_t N = c->plan.N;
  if (cudaMemcpyAsync(dst, c->acc + static_cast<uint64_t>(w) * N, N * sizeof(float), cudaMemcpyDeviceToDevice,
                      c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_set_residual(iwp_ctx* c, int32_t w, const float* src) {
  if (!c || !src || w < 0 || w >= c->plan.W) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  if (const int rc = flush_pending_zero(c)) return rc;
  const uint64_t N = c->plan.N;
  if (cudaMemcpyAsync(c->acc + static_cast<uint64_t>(w) * N, src, N * sizeof(float), cudaMemcpyDeviceToDevice,
                      c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_get_selection(iwp_ctx* c, int32_t w, uint32_t* idx, float* val) {
  if (!c || w < 0 || w >= c->plan.W) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  if (c->threshold_mode) {  // one list, the chosen node's; the whole capacity is copied
    if (w != c->leader) return IWP_ERR_INVALID;
    bool ok1 = true;
    if (idx)
      ok1 = ok1 && cudaMemcpyAsync(idx, c->sel_idx, c->list_cap * sizeof(uint32_t), cudaMemcpyDeviceToDevice,
                                   c->stream) == cudaSuccess;
    if (val)
      ok1 = ok1 && cudaMemcpyAsync(val, c->sel_val, c->list_cap * sizeof(float), cudaMemcpyDeviceToDevice,
                                   c->stream) == cudaSuccess;
    if (!ok1) {
      cudaGetLastError();
      return IWP_ERR_CUDA;
    }
    return IWP_OK;
  }
  const uint64_t K = c->plan.K;
  bool ok = true;
  if (idx)
    ok = ok && cudaMemcpyAsync(idx, c->sel_idx + static_cast<uint64_t>(w) * K, K * sizeof(uint32_t),
                               cudaMemcpyDeviceToDevice, c->stream) == cudaSuccess;
  if (val)
    ok = ok && cudaMemcpyAsync(val, c->sel_val + static_cast<uint64_t>(w) * K, K * sizeof(float),
                               cudaMemcpyDeviceToDevice, c->stream) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_get_mask(iwp_ctx* c, uint8_t* dst) {
  if (!c || !dst) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  const uint64_t N = c->plan.N, K = c->plan.K;
  if (cudaMemsetAsync(dst, 0, N, c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  if (c->leader < 0) return IWP_OK;
  if (c->threshold_mode) {
    k_thr_mask<<<148 * 8, THREADS, 0, c->stream>>>(c->sel_idx, c->d_list_len, static_cast<uint32_t>(c->list_cap), dst);
    if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
    return IWP_OK;
  }
  const unsigned blocks = static_cast<unsigned>((K + THREADS - 1) / THREADS);
  if (c->last_per_layer) {  // every layer's segment from its own chosen node's list
    k_layer_leader_sum_scatter<<<blocks, THREADS, 0, c->stream>>>(c->sel_idx, c->d_layers,
                                                                  static_cast<uint32_t>(c->plan.layers.size()), nullptr,
                                                                  nullptr, dst, N, K, c->plan.W, c->seed,
                                                                  static_cast<uint64_t>(c->t - 1));
    if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
    return IWP_OK;
  }
  for (int j = 0; j < c->last_chosen.n; ++j) {  // the index set is the union of the chosen nodes' lists
    k_mask_scatter<<<blocks, THREADS, 0, c->stream>>>(c->sel_idx + static_cast<uint64_t>(c->last_chosen.r[j]) * K, dst, K);
    if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  }
  return IWP_OK;
}

int iwp_encode_mask(iwp_ctx* c, const uint8_t* mask, uint8_t* bits) {
  if (!c || !mask || !bits) return IWP_ERR_INVALID;
  const uint64_t N = c->plan.N, n_bytes = (N + 7) / 8;
  k_pack_mask<<<static_cast<unsigned>((n_bytes + THREADS - 1) / THREADS), THREADS, 0, c->stream>>>(mask, bits, N);
  if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  return IWP_OK;
}

int64_t iwp_wire_mask_bytes(int64_t N) { return N < 0 ? -1 : ((N + 31) / 32) * 4; }

int iwp_wire_pack(iwp_ctx* c, const uint32_t* idx, int64_t n, uint8_t* bits) {
  if (!c || (!idx && n > 0) || !bits || n < 0 || (reinterpret_cast<uintptr_t>(bits) & 3u)) return IWP_ERR_INVALID;
  const uint64_t n_words = (c->plan.N + 31) >> 5;
  if (cudaMemsetAsync(bits, 0, n_words * sizeof(uint32_t), c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  c->launches += 1;
  if (n == 0) return IWP_OK;
  k_wire_pack<<<static_cast<unsigned>((static_cast<uint64_t>(n) + THREADS - 1) / THREADS), THREADS, 0, c->stream>>>(
      idx, static_cast<uint64_t>(n), reinterpret_cast<uint32_t*>(bits), c->plan.N, c->d_status);
  IWP_LAUNCH_CHECK(c);
  return IWP_OK;
}

int iwp_wire_unpack(iwp_ctx* c, const uint8_t* bits, uint32_t* idx, int64_t cap, int64_t* n_host) {
  if (!c || !bits || (!idx && cap > 0) || cap < 0 || (reinterpret_cast<uintptr_t>(bits) & 3u)) return IWP_ERR_INVALID;
  const uint64_t n_words = (c->plan.N + 31) >> 5;
  const unsigned chunks = static_cast<unsigned>((n_words + WIRE_CHUNK_WORDS - 1) / WIRE_CHUNK_WORDS);
  const uint32_t* words = reinterpret_cast<const uint32_t*>(bits);
  k_wire_count<<<chunks, THREADS, 0, c->stream>>>(words, n_words, c->d_wire_cnt);
  IWP_LAUNCH_CHECK(c);
  k_thr_scan<<<1, 1024, 0, c->stream>>>(c->d_wire_cnt, c->d_wire_off, chunks, c->d_wire_len);
  IWP_LAUNCH_CHECK(c);
  k_wire_expand<<<chunks, THREADS, 0, c->stream>>>(words, n_words, c->d_wire_off, idx, static_cast<uint64_t>(cap),
                                                  c->d_status);
  IWP_LAUNCH_CHECK(c);
  if (n_host) {
    uint32_t v = 0;
    if (cudaMemcpyAsync(&v, c->d_wire_len, sizeof(uint32_t), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
      cudaGetLastError();
      return IWP_ERR_CUDA;
    }
    *n_host = static_cast<int64_t>(v);
  }
  return IWP_OK;
}

int iwp_reset(iwp_ctx* c) {
  if (!c) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  const Sizes sz = sizes_of(c->plan, c->threshold_mode, c->list_cap);
  bool ok = cudaMemsetAsync(c->acc, 0, sz.acc, c->stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->zmask, 0, sz.zmask, c->stream) == cudaSuccess;
  c->zero_pending = false;
  ok = ok && cudaMemsetAsync(c->d_hist, 0, sz.hist, c->stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->d_reach, 0, sz.reach, c->stream) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->d_status, 0, sz.status, c->stream) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  if (c->threshold_mode && cudaMemsetAsync(c->d_list_len, 0, sizeof(uint32_t), c->stream) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  c->t = 0;
  c->leader = -1;
  return IWP_OK;
}

int iwp_set_option(iwp_ctx* c, const char* key, int64_t v) {
  if (!c || !key) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  if (!std::strcmp(key, "leader_override")) {
    if (v < -1 || v >= c->plan.W) return IWP_ERR_INVALID;
    c->leader_override = v;
    return IWP_OK;
  }
  if (!std::strcmp(key, "force_scalar")) {
    if (v != 0 && v != 1) return IWP_ERR_INVALID;
    c->force_scalar = v != 0;
    return IWP_OK;
  }
  if (!std::strcmp(key, "time_stages")) {
    if (v < 0 || v > 2) return IWP_ERR_INVALID;
    cudaStreamSynchronize(c->stream);
    stage_clear(c);
    c->time_stages = static_cast<int>(v);
    return IWP_OK;
  }
  if (!std::strcmp(key, "reserve_timed_steps")) {
    if (v < 0 || v > (1 << 20)) return IWP_ERR_INVALID;
    const size_t per_step = c->time_stages == 1 ? N_STAGES + 1 : 2;
    for (size_t i = 0; i < static_cast<size_t>(v) * per_step; ++i) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreate(&e) != cudaSuccess) {
        cudaGetLastError();
        return IWP_ERR_CUDA;
      }
      c->event_pool.push_back(e);
    }
    return IWP_OK;
  }
  if (!std::strcmp(key, "random_select")) {
    if (!c->threshold_mode || (v != 0 && v != 1)) return IWP_ERR_INVALID;
    c->random_select = v != 0;
    return IWP_OK;
  }
  if (!std::strcmp(key, "n_leaders")) {
    if (v < 1 || v > MAX_LEADERS || v > c->plan.W) return IWP_ERR_INVALID;
    c->n_leaders = static_cast<int32_t>(v);
    return IWP_OK;
  }
  if (!std::strcmp(key, "per_layer_leaders")) {
    if (c->threshold_mode || (v != 0 && v != 1)) return IWP_ERR_INVALID;
    c->per_layer_leaders = v != 0;
    return IWP_OK;
  }
  if (!std::strcmp(key, "leader_only_select")) {
    if (c->threshold_mode || (v != 0 && v != 1)) return IWP_ERR_INVALID;
    c->leader_only_select = v != 0;
    return IWP_OK;
  }
  if (!std::strcmp(key, "overlap")) {
    if (v != 0 && v != 1) return IWP_ERR_INVALID;
    c->overlap = static_cast<int>(v);
    return IWP_OK;
  }
  if (!std::strcmp(key, "pair_select")) {
    if (v < -1 || v > 1) return IWP_ERR_INVALID;
    c->pair_select = static_cast<int>(v);
    return IWP_OK;
  }
  if (!std::strcmp(key, "speculate")) {
    if (v != 0 && v != 1) return IWP_ERR_INVALID;
    c->speculate = v != 0;
    return IWP_OK;
  }
  return IWP_ERR_INVALID;
}

int iwp_get_stat(iwp_ctx* c, const char* key, int64_t* value) {
  if (!c || !key || !value) return IWP_ERR_INVALID;
  if (const int jrc = join_deferred(c)) return jrc;
  if (!std::strcmp(key, "launches")) {
    *value = c->launches;
    return IWP_OK;
  }
  if (!std::strcmp(key, "device_bytes")) {
    *value = static_cast<int64_t>(c->device_bytes);
    return IWP_OK;
  }
  if (!std::strcmp(key, "timed_steps")) {
    *value = static_cast<int64_t>(c->stage_events.size() / (N_STAGES + 1));
    return IWP_OK;
  }
  for (int st = 0; st < N_STAGES; ++st) {
    if (std::strcmp(key, kStageKeys[st])) continue;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) {
      cudaGetLastError();
      return IWP_ERR_CUDA;
    }
    double ns = 0.0;
    const size_t steps = c->stage_events.size() / (N_STAGES + 1);
    for (size_t i = 0; i < steps; ++i) {
      float ms = 0.f;
      cudaEvent_t e0 = c->stage_events[i * (N_STAGES + 1) + st], e1 = c->stage_events[i * (N_STAGES + 1) + st + 1];
      if (!e0 || !e1) continue;  // this boundary was not recorded in the current timing mode
      if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) {
        cudaGetLastError();
        return IWP_ERR_CUDA;
      }
      ns += static_cast<double>(ms) * 1e6;
    }
    *value = static_cast<int64_t>(ns);
    return IWP_OK;
  }
  if (!std::strcmp(key, "spec_pairs")) {
    *value = c->speculate ? c->spec_pairs : 0;
    return IWP_OK;
  }
  if (!std::strcmp(key, "spec_failed")) {
    *value = 0;
    if (!c->speculate || c->spec_pairs == 0 || c->info_clean) return IWP_OK;
    std::vector<PairInfo> h(c->n_pairs);
    if (cudaMemcpyAsync(h.data(), c->info_cur, h.size() * sizeof(PairInfo), cudaMemcpyDeviceToHost, c->stream) !=
            cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
      cudaGetLastError();
      return IWP_ERR_CUDA;
    }
    const int W = c->plan.W;
    for (uint32_t pr = 0; pr < c->n_pairs; ++pr) {
      const LayerDesc& L = c->plan.layers[c->plan.large_layers[pr / W]];
      if (L.sample == 0) continue;
      if (c->last_only >= 0 && static_cast<int>(pr % W) != c->last_only) continue;  // that worker made no selection
      const bool cand = h[pr].guess != GUESS_NONE && h[pr].total >= L.k && (h[pr].flags & 1u) == 0u;
      if (!cand) *value += 1;
    }
    return IWP_OK;
  }
  return IWP_ERR_INVALID;
}

}  // extern "C"

// =========================================================================================
// iwp_select_static: the exact top-k list of ONE layer for ONE worker without any allocation.
//
// Some callers must not allocate device memory while they run: code inside a memory-pool or
// arena discipline that forbids cudaMalloc after start-up, real-time loops where an allocation's
// implicit device synchronisation is unacceptable, or plug-ins that run under a host framework's
// "no allocation here" rule.  For them this entry point runs the same exact multi-pass select
// and stable compaction as the tiled path of iwp_step(), but takes every byte of scratch
// (histogram, select state, chunk tables and counts) from the fixed device array below instead
// of from a context created by iwp_create().
//
// The array's name is only a host-side handle; kernels get its device address, which is looked
// up once per device with cudaGetSymbolAddress() on the first call made with that device current.
// =========================================================================================
namespace {

constexpr int64_t STATIC_MAX_N = int64_t(1) << 24;  // largest layer the fixed scratch is sized for
constexpr uint32_t STATIC_CHUNK_ELEMS = CHUNK_TILES * TILE;
constexpr uint32_t STATIC_MAX_CHUNKS = static_cast<uint32_t>(STATIC_MAX_N / STATIC_CHUNK_ELEMS) + 1;

struct StaticScratch {
  uint32_t hist[NBINS];  // must be zero when a select starts
  uint2 state;
  PairInfo info;         // guess = none: the select reads the residual itself
  LayerDesc layer;
  uint32_t large_id;
  int status;
  uint2 chunk_cnt[STATIC_MAX_CHUNKS];
  Chunk chunks[STATIC_MAX_CHUNKS];
};

// Held by every GPU that loads this library, until the process exits (about 10 KB).
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int STATIC_MAX_DEVICES = 64;
StaticScratch* g_static_ptr[STATIC_MAX_DEVICES] = {};  // device address of the array, per device ordinal

// Fills the tables for a layer of n elements and clears what must start at zero.
__global__ void k_static_setup(StaticScratch* s, uint32_t n, uint32_t k, uint32_t n_chunks) {
  for (uint32_t b = threadIdx.x; b < NBINS; b += blockDim.x) s->hist[b] = 0;
  for (uint32_t j = threadIdx.x; j < n_chunks; j += blockDim.x) {
    Chunk c{};
    c.a = j * STATIC_CHUNK_ELEMS;
    c.len = (n - c.a < STATIC_CHUNK_ELEMS) ? n - c.a : STATIC_CHUNK_ELEMS;
    c.layer = 0;
    c.first_tile = 0;
    c.n_tiles = 0;
    c.first_chunk_of_layer = 0;
    s->chunks[j] = c;
    s->chunk_cnt[j] = make_uint2(0u, 0u);
  }
  if (threadIdx.x == 0) {
    s->state = make_uint2(0u, 0u);
    s->info = PairInfo{GUESS_NONE, 0u, 0u, 0u};
    LayerDesc L{};
    L.off = 0;
    L.n = n;
    L.k = k;
    L.koff = 0;
    L.large_index = 0;
    s->layer = L;
    s->large_id = 0;
    s->status = 0;
  }
}

template <bool VEC>
int run_select_static(StaticScratch* s, const float* residual, const float* weights, uint32_t n, uint32_t k, float eps,
                      uint32_t* idx, float* val, cudaStream_t st) {
  const uint32_t n_chunks = (n + STATIC_CHUNK_ELEMS - 1) / STATIC_CHUNK_ELEMS;
  k_static_setup<<<1, THREADS, 0, st>>>(s, n, k, n_chunks);
  if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  dim3 grid(n_chunks, 1);
  const WorkerSel all{WorkerSel::ALL, 0, -1};
  for (int pass = 0; pass < N_PASSES; ++pass) {
    k_hist<VEC, SEL_WARPS><<<grid, SEL_THREADS, 0, st>>>(residual, weights, s->chunks, &s->layer, &s->info, nullptr, nullptr, &s->state,
                                          s->hist, nullptr, nullptr, nullptr, eps, 0, 1, pass, n_chunks, all, nullptr);
    if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
    k_find_digit<SEL_WARPS><<<1, SEL_THREADS, 0, st>>>(&s->state, s->hist, &s->layer, &s->large_id, &s->info, nullptr, &s->status, 1, pass,
                                        all, nullptr);
    if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  }
  k_count<VEC><<<grid, SEL_THREADS, 0, st>>>(residual, weights, s->chunks, &s->layer, &s->info, nullptr, nullptr, &s->state,
                                         s->chunk_cnt, eps, 0, 1, n_chunks);
  if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  k_write<VEC, SEL_WARPS><<<grid, SEL_THREADS, 0, st>>>(residual, weights, s->chunks, nullptr, &s->layer, &s->info, nullptr, nullptr,
                                         nullptr, nullptr, &s->state, s->chunk_cnt, idx, val, nullptr, nullptr,
                                         &s->status, eps, 0, 0, 1, n_chunks, -1, all, nullptr, nullptr);
  if (cudaGetLastError() != cudaSuccess) return IWP_ERR_CUDA;
  return IWP_OK;
}

}  // namespace

extern "C" int iwp_select_static(const float* residual_dev, const float* weights_dev, int64_t n, double ratio, float eps,
                                 uint32_t* idx_dev, float* val_dev, int64_t* k_host, void* cuda_stream) {
  if (!residual_dev || !weights_dev || !idx_dev || !val_dev) return IWP_ERR_INVALID;
  if (n < 1 || n > STATIC_MAX_N) return IWP_ERR_INVALID;  // beyond what the fixed scratch is sized for
  if (!(eps > 0.f) || !std::isfinite(eps)) return IWP_ERR_INVALID;
  const int64_t k = keep_count(n, ratio);
  if (k < 1) return IWP_ERR_INVALID;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  if (!g_static_ptr[dev]) {  // first call with this device current: look up the array's device address
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return IWP_ERR_CUDA;
    }
    g_static_ptr[dev] = static_cast<StaticScratch*>(p);
  }
  if (k_host) *k_host = k;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool vec = aligned16(residual_dev) && aligned16(weights_dev);
  return vec ? run_select_static<true>(g_static_ptr[dev], residual_dev, weights_dev, static_cast<uint32_t>(n),
                                       static_cast<uint32_t>(k), eps, idx_dev, val_dev, st)
             : run_select_static<false>(g_static_ptr[dev], residual_dev, weights_dev, static_cast<uint32_t>(n),
                                        static_cast<uint32_t>(k), eps, idx_dev, val_dev, st);
}

extern "C" int iwp_select_static_status(int32_t* status_host, void* cuda_stream) {
  if (!status_host) return IWP_ERR_INVALID;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  if (!g_static_ptr[dev]) return IWP_ERR_INVALID;  // nothing has run on this device yet
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int v = 0;
  if (cudaMemcpyAsync(&v, &g_static_ptr[dev]->status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return IWP_ERR_CUDA;
  }
  *status_host = v;
  return IWP_OK;
}

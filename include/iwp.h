/*
 * iwp.h - C ABI of the importance-weighted gradient pruning step for data-parallel
 *         all-reduce (arXiv 1901.01544), for W simulated workers held in one GPU.
 *
 * One call of iwp_step() performs, for every worker w and every layer l
 * (Algorithm 1 of the paper; Section 3.2 "Importance Weighted Pruning"):
 *   (a) residual accumulation        acc[w][i] += grads[w][i]
 *   (b) gradient importance          imp = |acc[w][i]| / (|weights[i]| + eps)
 *   (c) layer-wise selection         the k_l = ceil(n_l / ratio) elements with the largest
 *                                    importance (ties: lower index first) - Algorithm 1's
 *                                    "Mask <- |grad / w| > thr" with thr = k_l-th largest
 *   (d) sparse encoding              ascending (index, value) lists per worker
 *   (e) index agreement              one seeded-randomly chosen worker ("choose random node")
 *                                    supplies the index set S every worker gathers at
 *   (f) reduction                    update[S] = sum over workers in ascending worker order
 *                                    (the ring all-reduce of the masked gradients), 0 elsewhere
 *   (g) local accumulation           acc[w][S] = 0 for every w; everything else stays
 *
 * All arithmetic is IEEE-754 binary32, round to nearest even, no fused multiply-add,
 * denormals kept.  Inputs must be finite.  Indices are 32-bit flat element offsets.
 *
 * Conventions
 *   - every function returns an int status (IWP_OK = 0, errors negative); nothing throws,
 *     aborts or prints; device code never traps or asserts (errors end up in a status word
 *     read by iwp_sync_status()).
 *   - pointers named *_dev are DEVICE pointers, *_host are HOST pointers; the caller owns
 *     every buffer it passes in; the library owns what it allocates in iwp_create().
 *   - one context = one CUDA device = one stream = one caller thread at a time.
 *   - the library needs a CUDA device; there is no CPU fallback.
 */
#ifndef IWP_H_
#define IWP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct iwp_ctx iwp_ctx;

enum {
  IWP_OK = 0,
  IWP_ERR_INVALID = -1,  /* bad argument (NULL, size, range, alignment of a typed pointer) */
  IWP_ERR_OOM = -2,      /* device or host allocation failed */
  IWP_ERR_CUDA = -3,     /* a CUDA runtime call or kernel launch failed */
  IWP_ERR_INTERNAL = -4, /* a device-side conservation check failed (counts do not add up) */
  IWP_ERR_TIMEOUT = -5,  /* a bounded device-side wait gave up (unused: no kernel here waits) */
  IWP_ERR_CAPACITY = -6  /* threshold mode: the index set did not fit the list (see iwp_create_threshold) */
};

/* Human-readable name of a status code; never NULL. */
const char* iwp_strerror(int status);

/* ---- pure host helpers (no GPU needed) --------------------------------------------- */

/* Keep count of a layer of n elements at compression ratio R (Table 1 of the paper quotes
 * ratios of 64x and 58.8x): ceil(n / R) in double precision, clamped to [1, n].
 * Returns 0 for invalid input (n < 1, R < 1 or not finite). */
int64_t iwp_keep_count(int64_t n, double ratio);

/* The worker that supplies the index set at step t (0-based) - Section 3.2's randomly
 * chosen node.  The paper names no generator; this one is
 *   ((mix64(seed + (t + 1) * 0x9E3779B97F4A7C15) >> 32) * W) >> 32
 * with the splitmix64 finaliser as mix64.  Returns -1 if W < 1. */
int32_t iwp_leader_at(uint64_t seed, uint64_t t, int32_t W);

/* The chosen node of layer `layer` (0-based) at step t when every layer draws its own (option
 * "per_layer_leaders"; Algorithm 1 draws the node inside its loop over layers):
 * ((mix64(seed + (t+1)*0x9E3779B97F4A7C15 + (layer+1)*0xA0761D6478BD642F) >> 32) * W) >> 32.
 * Host-only helper; -1 for W < 1 or layer < 0. */
int32_t iwp_layer_leader_at(uint64_t seed, uint64_t t, int32_t layer, int32_t W);

/* The n distinct chosen nodes r_1..r_n of step t (Algorithm 1: "choose random node r_1, r_2, ... r_n"), drawn
 * without replacement: u_j = ((mix64(seed + (t+1)*0x9E3779B97F4A7C15 + j*0xD1B54A32D192ED03) >> 32) * (W-j)) >> 32
 * picks the u_j-th of the workers not chosen yet; out_host[0] equals iwp_leader_at().  1 <= n <= min(W, 8).
 * Errors: IWP_ERR_INVALID. */
int iwp_leaders_at(uint64_t seed, uint64_t t, int32_t W, int32_t n, int32_t* out_host);

/* Sizes the planner derives from a layer list, without touching a GPU.
 * out[0] = N (total elements)            out[1] = K (total keep count per worker)
 * out[2] = layers on the one-CTA path    out[3] = layers on the tiled path
 * out[4] = tiles                          out[5] = chunks
 * out[6] = device bytes iwp_create() would allocate
 * out[7] = 1 if 128-bit vector access is possible for library-owned buffers (N % 4 == 0)
 * Returns IWP_ERR_INVALID under the same rules as iwp_create(). */
int iwp_plan_sizes(const int64_t* layer_sizes_host, int32_t n_layers, int32_t W, double ratio, int64_t out[8]);

/* ---- life cycle -------------------------------------------------------------------------- */

/* Creates a context on the CURRENT CUDA device.
 *   layer_sizes_host  n_layers element counts; every tensor is its own selection unit
 *                     (Algorithm 1 loops over layers j = 0..M); copied, caller keeps ownership
 *   W                 number of simulated workers (the paper's N nodes), 1 .. 65535
 *   ratio             compression factor R >= 1 (64 keeps 1/64 of each layer), finite
 *   eps               guard added to |weight| in the importance; > 0 and finite
 *   seed              seed of the leader draw
 * Allocates and zeroes the residuals acc[W][N] plus select scratch and the (index, value)
 * lists.  Errors: IWP_ERR_INVALID (NULL, n_layers < 1, a size < 1, W out of range, bad ratio or eps,
 * N >= 2^32), IWP_ERR_OOM, IWP_ERR_CUDA; *out is NULL on error. */
int iwp_create(iwp_ctx** out, const int64_t* layer_sizes_host, int32_t n_layers, int32_t W, double ratio, float eps,
               uint64_t seed);

/* Absolute-threshold mode: Algorithm 1 of the paper as printed.  Per step, only the chosen node r forms a
 * mask, layer by layer, Mask_r = |acc_r / w| > thr[layer] (strict, with the eps guard in the denominator);
 * its index set S has whatever size results; every node then contributes acc[w][S] to the ordered sum,
 * update[S] = sum, and acc[w][S] = 0.  No other worker makes a selection of its own.  The paper used
 * thresholds of 0.005 ... 0.1 (Section 4.1).
 *   max_list   capacity of the index list in entries; 0 or anything above N means N.  If a step's index
 *              set is longer, IWP_ERR_CAPACITY is raised in the status word and that step's update is
 *              incomplete.
 * A context created here takes iwp_set_thresholds() before its first step; iwp_get_selection() is valid for
 * the last step's leader only and copies max_list entries of which the first iwp_get_list_length() are
 * meaningful; iwp_get_layout() reports keep counts of 0.  Same errors as iwp_create(). */
int iwp_create_threshold(iwp_ctx** out, const int64_t* layer_sizes_host, int32_t n_layers, int32_t W, float eps,
                         uint64_t seed, int64_t max_list);

/* n_layers thresholds (host array, copied), each >= 0; +inf sends nothing from that layer.  Synchronises
 * the stream.  Errors: IWP_ERR_INVALID (NULL, not a threshold-mode context, negative or NaN value). */
int iwp_set_thresholds(iwp_ctx* ctx, const float* thr_host);

/* Section 3.4, layer-wise threshold (Eq. 4; its two printed branches carry the same condition and are
 * read as "v > C" and "otherwise"): with on = 1 every following step of a threshold-mode context derives,
 * for each chosen node and layer, thr = alpha + beta * v if v > c_split else alpha - beta * v, where
 * v = var / mean of the layer's importances on that node, and uses it in place of the fixed thresholds
 * (iwp_set_thresholds() is then not needed).  So that the value depends on no summation order,
 * S1 = sum imp and S2 = sum imp^2 are exact sums rounded once to binary64; then, one binary64 operation
 * at a time, mean = S1 / n, var = S2 / n - mean * mean, v = var / mean (0 when mean is 0); thr is rounded
 * to binary32, -0 taken as +0; a negative thr selects the whole layer.  on = 0 returns to the fixed
 * thresholds.  Errors: IWP_ERR_INVALID (NULL, not a threshold-mode context, non-finite parameter). */
int iwp_set_layerwise(iwp_ctx* ctx, int32_t on, double alpha, double beta, double c_split);

/* The thresholds the last layer-wise step derived: n_chosen rows (r_1 first) of one float per layer to
 * dst_dev (room for 8 rows), the number of rows to *n_chosen_host (0 before the first such step).
 * Asynchronous on the context's stream.  IWP_ERR_INVALID unless iwp_set_layerwise() is on. */
int iwp_get_layer_thresholds(iwp_ctx* ctx, float* dst_dev, int32_t* n_chosen_host);

/* Number of entries of the last step's index set (threshold mode: synchronises the stream and reads
 * it from the device; ratio mode: K). */
int iwp_get_list_length(iwp_ctx* ctx, int64_t* len_host);

/* Synchronises the context's stream and frees everything iwp_create() allocated.
 * NULL is a no-op returning IWP_OK. */
int iwp_destroy(iwp_ctx* ctx);

/* Stream all later work of this context is enqueued on (a cudaStream_t passed as void*;
 * NULL = the legacy default stream, which is also the initial setting). */
int iwp_set_stream(iwp_ctx* ctx, void* cuda_stream);

/* Momentum on the locally kept residual (Eq. 3 of the paper: s_t = sparse(m g_{t-1} + g_t)): step (a)
 * becomes acc[w][i] = m * acc[w][i] + grads[w][i], one rounded product then one rounded sum.
 * m = 1 (the default) is the plain accumulation of Section 3.2; m = 0 forgets what was not sent.
 * Takes effect from the next step.  Errors: IWP_ERR_INVALID (NULL, m negative or not finite). */
int iwp_set_momentum(iwp_ctx* ctx, float m);

/* ---- the step ---------------------------------------------------------------------------- */

/* One pruned all-reduce step, steps (a)-(g) above (Algorithm 1, one iteration of the loop over t
 * without the optimizer update, which stays with the caller).
 *   grads_dev    W*N floats, worker-major with stride N, layers concatenated without padding;
 *                read only
 *   weights_dev  N floats, one copy shared by all workers (synchronous replicas, Eq. 1); read only
 *   update_dev   N floats, fully overwritten: +0 outside the index set, the ordered worker sum
 *                inside; must not alias the other two
 * Asynchronous: enqueues kernels on the context's stream and returns without synchronising;
 * the three buffers must stay valid until the stream has run the step, after which the caller may
 * change or free them.  When the stream has run the step, update_dev and the residuals are final.
 * The (index, value) lists of workers other than the leader, which nothing in the step consumes,
 * may still be in the making on streams of the library's own (option "overlap"); they read library
 * memory only, and every accessor, iwp_sync_status() and the next step order themselves after them.
 * 128-bit accesses are used when N % 4 == 0 and all three pointers are 16-byte aligned, scalar
 * accesses otherwise.
 * Advances the step counter.  Errors: IWP_ERR_INVALID (NULL), IWP_ERR_CUDA (launch failure). */
int iwp_step(iwp_ctx* ctx, const float* grads_dev, const float* weights_dev, float* update_dev);

/* ---- workers spread over several contexts (one context per GPU) ------------------------------
 * The paper's deployment is a ring of nodes: the chosen node's index set travels to everybody
 * (Algorithm 1: AllGather of the encoded mask), then the masked gradients are all-reduced.  With the W
 * workers of a job split into consecutive groups, one context of W_local workers per group, a step is
 *   1. iwp_shard_select() on every context: steps (a)-(d) for its own workers;
 *   2. the caller reads the chosen worker's list from the context that holds it
 *      (iwp_get_selection(), K indices) and sends it to every context (broadcast);
 *   3. iwp_shard_gather() on every context: its workers' residuals at those indices (step (e));
 *   4. the caller concatenates the groups' values in global worker order (all-gather);
 *   5. iwp_shard_apply() on every context: step (f) over all W workers in ascending order - so every
 *      context holds the same update, bit for bit the one a single context of W workers computes -
 *      and step (g) for its own workers.
 * The transport (steps 2 and 4) is the caller's: the Python binding's ShardedPruner uses
 * torch.distributed (NCCL).  Ratio-mode contexts only; all three calls are asynchronous on the
 * context's stream like iwp_step(). */

/* Steps (a)-(d) for this context's W_local workers.  update_dev (N floats) is zero-filled here and
 * must be the buffer later given to iwp_shard_apply().  Does not advance the step counter. */
int iwp_shard_select(iwp_ctx* ctx, const float* grads_dev, const float* weights_dev, float* update_dev);

/* vals_dev[w * n + j] = residual of local worker w at idx_dev[j], w < W_local, j < n (the values as they
 * are after iwp_shard_select()).  idx_dev: n distinct flat indices below N. */
int iwp_shard_gather(iwp_ctx* ctx, const uint32_t* idx_dev, int64_t n, float* vals_dev);

/* update_dev[idx_dev[j]] = +0 + (((v[0][j] + v[1][j]) + v[2][j]) + ...) over the W_total rows of
 * vals_all_dev (row w = global worker w, n floats each); the residuals of this context's workers
 * become +0 at the n indices.  Advances the step counter.  IWP_ERR_INVALID if W_total < W_local. */
int iwp_shard_apply(iwp_ctx* ctx, const uint32_t* idx_dev, int64_t n, const float* vals_all_dev, int32_t W_total,
                    float* update_dev);

/* The same step with HOST buffers (pinned memory recommended): copies grads and weights to
 * library-owned staging buffers (allocated on first use), runs iwp_step(), copies the update
 * back and synchronises the stream before returning. */
int iwp_step_host(iwp_ctx* ctx, const float* grads_host, const float* weights_host, float* update_host);

/* Makes the context's stream wait for everything the last step left running on the library's own side
 * streams (with the overlapped schedule the selects of workers other than the chosen node, whose lists
 * no step consumes, outlive iwp_step()).  Nothing is synchronised with the host: after this call, work
 * enqueued on the context's stream - an event record, a copy - is ordered behind ALL of the step's
 * kernels.  Every accessor does this by itself.  Errors: IWP_ERR_INVALID, IWP_ERR_CUDA. */
int iwp_join(iwp_ctx* ctx);

/* Synchronises the stream and returns the device status word: IWP_OK, IWP_ERR_INTERNAL
 * (a count check failed inside a kernel; results of that step are undefined) or IWP_ERR_CUDA. */
int iwp_sync_status(iwp_ctx* ctx);

/* ---- state, accessors (none of these is on the timed path) ------------------------------- */

/* off_host[l] = flat offset of layer l, k_host[l] = its keep count; either may be NULL. */
int iwp_get_layout(iwp_ctx* ctx, int64_t* off_host, int64_t* k_host);
/* out[0] = N, out[1] = K, out[2] = n_layers, out[3] = W. */
int iwp_get_sizes(iwp_ctx* ctx, int64_t out[4]);
int iwp_get_step(iwp_ctx* ctx, int64_t* t_host);
int iwp_set_step(iwp_ctx* ctx, int64_t t); /* checkpoint / resume; t >= 0 */
/* Leader used by the last step (-1 before the first). */
int iwp_get_leader(iwp_ctx* ctx, int32_t* leader_host);
/* Residual acc[w][0..N) copied to / from a device buffer of N floats (stream-ordered). */
int iwp_get_residual(iwp_ctx* ctx, int32_t w, float* dst_dev);
int iwp_set_residual(iwp_ctx* ctx, int32_t w, const float* src_dev);
/* Worker w's list of the last step: K ascending global indices (layer segments of k_l entries
 * in layer order) and the accumulated values at those indices as they were BEFORE step (g)
 * zeroed what was sent.  Device buffers of K entries; either may be NULL. */
int iwp_get_selection(iwp_ctx* ctx, int32_t w, uint32_t* idx_dev, float* val_dev);
/* Algorithm 1's encode_uint8(Mask): N bytes on the device, 1 where the element is in the
 * last step's index set, else 0. */
int iwp_get_mask(iwp_ctx* ctx, uint8_t* dst_dev);

/* The other reading of Algorithm 1's encode_uint8(Mask): eight elements per byte.  mask_dev: N bytes as
 * written by iwp_get_mask(); bits_dev: (N + 7) / 8 bytes, bit i % 8 of byte i / 8 = mask_dev[i] != 0.
 * Asynchronous on the context's stream; an accessor, not on the timed path (the path itself carries the
 * sorted index list). */
int iwp_encode_mask(iwp_ctx* ctx, const uint8_t* mask_dev, uint8_t* bits_dev);

/* ---- wire formats of the index set (workers spread over GPUs) ------------------------------- */

/* Algorithm 1 sends the index set as AllGather(encode_uint8(Mask)) ahead of the all-reduce of the masked
 * gradients.  Two encodings are offered to whoever moves the bytes: the sorted uint32 index list (4 bytes
 * per entry - what iwp_get_selection() returns) and the mask at one bit per element, bit i % 8 of byte
 * i / 8, padded to whole 32-bit words.  The list is the shorter one when the set holds fewer than N / 32
 * entries (compression above 32), the mask otherwise. */

/* Bytes of the one-bit-per-element mask of an N-element job: 4 * ceil(N / 32).  Pure host function. */
int64_t iwp_wire_mask_bytes(int64_t N);
/* idx_dev[0..n) (element indices < N, any order, no duplicates needed) -> bits_dev (iwp_wire_mask_bytes(N)
 * bytes, 4-byte aligned, fully overwritten; idx_dev may be NULL when n = 0).  Asynchronous on the context's stream.  An index >= N sets the
 * status word to IWP_ERR_INTERNAL and is skipped. */
int iwp_wire_pack(iwp_ctx* ctx, const uint32_t* idx_dev, int64_t n, uint8_t* bits_dev);
/* bits_dev -> the ascending index list in idx_dev[0..cap).  Asynchronous on the context's stream; with
 * n_host != NULL the call waits for the stream and stores the number of set bits there.  More set bits
 * than cap: the surplus is dropped and the status word becomes IWP_ERR_CAPACITY. */
int iwp_wire_unpack(iwp_ctx* ctx, const uint8_t* bits_dev, uint32_t* idx_dev, int64_t cap, int64_t* n_host);

/* acc <- 0, step counter <- 0, status word <- 0. */
int iwp_reset(iwp_ctx* ctx);

/* The same with the copies of consecutive calls overlapped: the call enqueues the host-to-device copies on a
 * copy stream of the library's own, the step on the context's stream and the copy of the update to
 * update_host on a second copy stream, and returns without waiting.  Two staging sets are used in turn, so
 * the inputs of call k + 1 travel while step k runs and while update k travels the other way.  The host
 * buffers of a call must stay untouched until iwp_host_wait() (pinned memory is needed for the copies to
 * overlap at all); update_host of call k is valid after iwp_host_wait() or once call k + 2 has returned
 * and the context's stream has reached it.  Same errors as iwp_step_host(). */
int iwp_step_host_async(iwp_ctx* ctx, const float* grads_host, const float* weights_host, float* update_host);

/* Blocks until every iwp_step_host_async() call made so far has delivered its update. */
int iwp_host_wait(iwp_ctx* ctx);

/* Options (tests and experiments):
 *   "leader_override"  >= 0 forces the leader of every following step, -1 = seeded draw
 *   "force_scalar"     1 = never use 128-bit accesses
 *   "n_leaders"        1 .. min(W, 8) chosen nodes per step, drawn without replacement, whose index sets are
 *                      OR-ed (Algorithm 1: Mask = OR Mask_ri).  Threshold mode: the masks of the chosen
 *                      nodes; the listed values are r_1's.  Ratio mode: the union of the chosen nodes' own
 *                      top-k lists (every worker still lists its own top-k; iwp_get_mask() gives the union).
 *                      A forced leader ("leader_override") makes the step a one-node step
 *   "per_layer_leaders" ratio-mode contexts only: 1 = every layer draws its own chosen node each step
 *                      (iwp_layer_leader_at()); the index set is, layer by layer, that node's list segment.
 *                      Ignored while a leader is forced or several chosen nodes are set.  0 (default) = one
 *                      node per step for all layers
 *   "random_select"    threshold-mode contexts only: 1 = Section 3.3's random gradient selection: an
 *                      element whose importance does not exceed its layer's threshold is still sent iff
 *                      u < importance / thr (fp32 quotient), u = u24 * 2^-24 with
 *                      u24 = mix64(seed + (t+1)*0x9E3779B97F4A7C15 + (i+1)*0xC2B2AE3D27D4EB4F) >> 40
 *                      for element i at step t; 0 (default) = off
 *   "leader_only_select" ratio-mode contexts only: 1 = only the chosen node of a step selects and lists
 *                      (Algorithm 1 consumes no other worker's index set); update, the chosen node's list,
 *                      mask and every residual are those of the default; iwp_get_selection() of any other
 *                      worker then returns unspecified contents.  Ignored with several chosen nodes, with
 *                      "per_layer_leaders" and in the sharded phases.  0 (default) = every worker lists
 *                      its own top-k
 *   "speculate"        1 (default) = sample-based threshold guess so that large layers are
 *                      read once; 0 = always the multi-pass exact select.  Both are exact.
 *   "pair_select"      1 = on the single-read path, layers of at most 640 tiles (2.6 M elements) are selected
 *                      and listed by one kernel launch with one thread-block cluster per (layer, worker)
 *                      pair; 0 = every tiled layer goes through the chain of histogram, digit and compaction
 *                      launches; -1 (default) = the library decides at create: the cluster launch for small
 *                      jobs (at most 64 pairs, no larger layer), where it is faster.  Same results either way.
 *   "overlap"          1 = the leader's select runs beside the other workers' streaming pass and the
 *                      other workers' selects beside the reduction and the head of the next step;
 *                      0 = every kernel of a step in one sequence.  Same results either way; the
 *                      default is 1 when the tiled layers hold at least 2^25 elements over all
 *                      workers (below that the extra launches cost more than they hide), else 0.
 *   "time_stages"      1 = record a CUDA event at every stage boundary of each following step
 *                      (read the totals with iwp_get_stat; steps run as with "overlap" 0 meanwhile);
 *                      2 = only before and after the dominant streaming stage (two events per step);
 *                      0 = stop and discard them
 *   "reserve_timed_steps" n: creates the CUDA events of the next n timed steps now (in the current
 *                      "time_stages" mode), so that a timed step only records them
 * Unknown key or out-of-range value: IWP_ERR_INVALID. */
int iwp_set_option(iwp_ctx* ctx, const char* key, int64_t value);

/* Counters: "launches" (kernels and memsets enqueued since create), "device_bytes",
 * "spec_pairs" / "spec_failed" ((worker, layer) pairs that tried / fell back from the
 * single-read path in the last step; reading them synchronises the stream).
 * With "time_stages" on: "timed_steps" and the summed device time in nanoseconds of each
 * stage over those steps - "time_small_ns" (one-CTA path), "time_sample_ns" (threshold
 * guess from a sample), "time_accumulate_ns" (step (a) on the
 * tiled path), "time_select_ns" (c), "time_compact_ns" (d), "time_gather_ns" ((e)-(g)).
 * Unknown key: IWP_ERR_INVALID. */
int iwp_get_stat(iwp_ctx* ctx, const char* key, int64_t* value_host);

/* ---- selection without any allocation --------------------------------------------------- */

/* (No counterpart in the paper: this entry point exists for callers of this library that are not
 * allowed to allocate device memory while they run - code under a start-up-only arena or pool
 * discipline, latency-critical loops that cannot afford the device synchronisation an allocation
 * implies, plug-ins bound by a host framework's no-allocation rule.)
 *
 * Writes the exact top-k list of ONE layer for ONE worker: the k = ceil(n / ratio) elements of
 * residual_dev[0..n) with the largest importance |residual| / (|weights| + eps), ties to the lower
 * index, as ascending indices idx_dev[0..k) and their residual values val_dev[0..k) - the same
 * result, bit for bit, as the list iwp_step() builds for that layer.  It needs no context and
 * calls no cudaMalloc / cudaFree or any other allocating routine: all scratch lives in a fixed
 * device array of about 10 KB that every GPU loading this library holds until the process exits.
 *
 *   residual_dev, weights_dev  n floats each, device, read only
 *   n                          1 .. 16 777 216 (2^24); larger layers are rejected with IWP_ERR_INVALID
 *   ratio, eps                 as in iwp_create()
 *   idx_dev, val_dev           device buffers of at least k entries, overwritten
 *   k_host                     optional: receives k
 *   cuda_stream                stream the kernels are enqueued on (NULL = legacy default stream)
 *
 * Asynchronous like iwp_step().  The first call made with a given device current looks up the
 * scratch array's device address; make that first call before any stream capture begins.  All
 * calls on a device share the one scratch array (it keeps the previous call's contents; the entry
 * point clears what must start at zero), so two calls whose kernels can overlap on the GPU - on
 * different streams, or from different threads - race: serialise them.
 * Errors: IWP_ERR_INVALID (NULL pointer, n out of range, bad ratio or eps), IWP_ERR_CUDA.  The return
 * value covers the arguments and the launches only; the kernels' own count checks (they fail on
 * non-finite inputs or when two calls raced) are read back with iwp_select_static_status(). */
int iwp_select_static(const float* residual_dev, const float* weights_dev, int64_t n, double ratio, float eps,
                      uint32_t* idx_dev, float* val_dev, int64_t* k_host, void* cuda_stream);

/* Device status word of the last iwp_select_static() call on the current device: copies it to
 * *status_host behind everything enqueued on cuda_stream and waits for that stream.  0, or
 * IWP_ERR_INTERNAL when a count check of the select or the compaction failed (the list is then not to be
 * trusted).  Allocates nothing.  Errors: IWP_ERR_INVALID (NULL pointer, or no call was made on this
 * device yet), IWP_ERR_CUDA. */
int iwp_select_static_status(int32_t* status_host, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* IWP_H_ */

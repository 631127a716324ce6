/* gorgo.h -- C ABI of libgorgo_b200: batched replay of a population of GORGO routing
 * cost-model parameter vectors over one request trace on one NVIDIA B200 (sm_100a).
 *
 * The operation (paper Section 2.2, Eq. 1-3; Section 2.3): for every candidate parameter
 * vector and every request of the trace, in trace order, compute on every replica the
 * longest cached prefix of the request's 512-token blocks, the score
 *     cost_i = ((w_net * RTT[origin][i]) + (w_prefill * uncached_tokens_i)) + (w_queue * q_i)
 * with q_i the proxy-recorded in-flight input tokens of replica i (optionally times a
 * per-replica normaliser), route to the lowest-index argmin, update that replica's LRU block
 * cache and its slot/queue state under the deterministic service model below, and record
 * TTFT = network + queue wait + prefill of the uncached tokens (Eq. 1) and the end-to-end
 * latency.  Each candidate's latencies are reduced to their 95th percentile (nearest rank),
 * the objective the paper tunes (Section 4).
 *
 * Service model (the paper names the need for one in Section 2.1 but gives none): S slots per
 * replica; a request arrives at the engine RTT after its scaled timestamp, takes the slot that
 * frees first, prefills `prefill_ms_per_token` x uncached tokens, then decodes
 * `tpot_ms` x max(output_tokens-1, 0); it counts as in flight at the proxy until it finishes.
 * The cache learns a request at dispatch; eviction is LRU by (request index, block position),
 * deepest block of the oldest request first.  All cost and time arithmetic is IEEE fp64,
 * round-to-nearest, no fused multiply-add, in the order written above.
 *
 * Conventions: every function returns GORGO_OK (0) or a negative gorgo_status.  No function
 * throws, aborts or prints.  Pointers are HOST pointers unless the comment says DEVICE.  The
 * library never allocates or frees device memory: the caller supplies every device buffer
 * (256-byte aligned) and keeps it alive while the handle uses it.  `cuda_stream` is a
 * cudaStream_t passed as void* (NULL = the default stream); work is enqueued on it and, unless
 * stated otherwise, the call does not wait for it.  A handle may be used by one host thread at
 * a time; distinct handles are independent.
 */
#ifndef GORGO_H_
#define GORGO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gorgo_sim gorgo_sim_t;

typedef enum gorgo_status {
  GORGO_OK = 0,
  GORGO_ERR_INVALID_ARG = -1,         /* NULL pointer, zero size, value out of the stated range   */
  GORGO_ERR_BAD_TRACE = -2,           /* trace violates a precondition listed at gorgo_trace_upload */
  GORGO_ERR_NONFINITE_PARAM = -3,     /* NaN/Inf among the cost-model parameters or the time scale */
  GORGO_ERR_WORKSPACE_TOO_SMALL = -4, /* a caller-supplied device buffer is smaller than required  */
  GORGO_ERR_CUDA = -5,                /* a CUDA runtime call failed                                */
  GORGO_ERR_DEVICE_LIMIT = -6,        /* a bounded device loop hit its limit (internal invariant)  */
  GORGO_ERR_NO_TRACE = -7,            /* the call needs an uploaded trace                          */
  GORGO_ERR_OUT_OF_ORDER = -8,        /* gorgo_route_batch: `first` is not the next request        */
  GORGO_ERR_STATIC_LIMIT = -9         /* gorgo_eval_population_static: trace too large for the     */
                                      /* library's built-in scratch array                          */
} gorgo_status;

/* Simulator configuration; copied by gorgo_sim_create (rtt_ms included). */
typedef struct gorgo_config {
  uint32_t n_replicas;          /* R, 1..64                                                      */
  uint32_t n_regions;           /* G >= 1, origin regions of requests; G*R <= 4096               */
  uint32_t slots_per_replica;   /* S, 1..65535 (paper: max_concurrent_requests = 64, Section 4)   */
  uint32_t block_tokens;        /* B >= 1 tokens per cache block (512)                            */
  uint64_t cache_blocks;        /* C >= 1 blocks per replica                                      */
  uint32_t n_params;            /* K: 3 = (w_net, w_prefill, w_queue), or 3 + R with per-replica  */
                                /* queue-load normalisers appended                                */
  uint32_t reserved;            /* must be 0                                                      */
  double prefill_ms_per_token;  /* finite, >= 0                                                   */
  double tpot_ms;               /* finite, >= 0: time per output token after the first            */
  const double *rtt_ms;         /* G*R row-major [origin][replica], finite, >= 0                  */
  int32_t device;               /* CUDA device ordinal                                            */
} gorgo_config_t;

/* Section 2.2 (signals of Eq. 2): creates a simulator for one replica fleet. */
int gorgo_sim_create(const gorgo_config_t *cfg, gorgo_sim_t **out);
int gorgo_sim_destroy(gorgo_sim_t *sim);

/* Upper bound of the device bytes gorgo_trace_upload needs for a trace of `n_requests`
 * requests with `n_block_ids` block ids in total. */
int gorgo_trace_bytes(uint64_t n_requests, uint64_t n_block_ids, uint64_t *bytes_out);

/* Section 3 (Mooncake-format trace: timestamps plus request metadata).  Validates the host
 * arrays, renumbers block ids to dense 32-bit numbers (only equality of ids matters), builds
 * the per-occurrence "next occurrence of the same block" links used by the LRU, and copies
 * everything into `dev_trace_buf` (DEVICE, caller-owned, must stay alive and untouched while the
 * trace is in use).  Waits for the copy, so the host arrays may be freed on return.
 * Preconditions (else GORGO_ERR_BAD_TRACE): 1 <= n_requests < 2^32-1; ts_ms finite, >= 0 and
 * non-decreasing; hash_off[0] = 0, non-decreasing, hash_off[n] < 2^32-1;
 * blocks of request r = hash_off[r+1]-hash_off[r] = ceil(input_tokens[r]/B) <= min(C, 65535);
 * no id twice inside one request; origin[r] < G (origin may be NULL = all 0). */
int gorgo_trace_upload(gorgo_sim_t *sim, uint64_t n_requests, const double *ts_ms,
                       const uint32_t *input_tokens, const uint32_t *output_tokens,
                       const uint16_t *origin, const uint64_t *hash_off,
                       const uint64_t *hash_ids, void *dev_trace_buf, uint64_t dev_trace_bytes,
                       void *cuda_stream);

/* Online boundary (Section 2.3: the proxy routes requests as they arrive): a trace that grows.
 * gorgo_trace_begin lays `dev_trace_buf` (DEVICE, >= gorgo_trace_bytes(max_requests,
 * max_block_ids) bytes, 256-byte aligned) out for up to `max_requests` requests with up to
 * `max_block_ids` block ids in total and forgets any earlier trace of the handle.
 * gorgo_trace_append adds `n_requests` >= 1 requests after the ones already there; the arguments
 * are those of gorgo_trace_upload for the new requests alone (`hash_off` starts at 0; `ts_ms`
 * continues non-decreasing from the last request so far).  The copies are enqueued on
 * `cuda_stream`, ordered after earlier batches on the same stream; the call returns when the
 * host arrays may be reused.  Returns GORGO_ERR_WORKSPACE_TOO_SMALL when a capacity would be
 * exceeded and GORGO_ERR_BAD_TRACE for a violated precondition; in both cases the trace is as
 * it was before the call.  GORGO_ERR_NO_TRACE without a preceding gorgo_trace_begin (a trace
 * given to gorgo_trace_upload cannot grow).
 *   Once the first batch is in, every call that takes a trace works on the requests appended so
 * far.  Workspace and state sizes (gorgo_workspace_bytes, gorgo_state_bytes) are computed for
 * the capacities, so a persistent state set up by gorgo_sim_reset stays valid while the trace
 * grows: gorgo_route_batch may route requests that were not known when the state was reset or
 * when earlier batches ran.  Routing appended requests batch by batch gives bit for bit what
 * routing the whole trace at once gives (a request still in flight at the end of the known
 * trace is kept in the state and leaves the queue signal of Eq. 2 at the first appended request
 * that arrives at or after its finish time); use one time scale from reset on. */
int gorgo_trace_begin(gorgo_sim_t *sim, uint64_t max_requests, uint64_t max_block_ids,
                      void *dev_trace_buf, uint64_t dev_trace_bytes);
int gorgo_trace_append(gorgo_sim_t *sim, uint64_t n_requests, const double *ts_ms,
                       const uint32_t *input_tokens, const uint32_t *output_tokens,
                       const uint16_t *origin, const uint64_t *hash_off, const uint64_t *hash_ids,
                       void *cuda_stream);

/* Facts about the uploaded trace: requests, block ids in total, distinct block ids. */
int gorgo_trace_info(const gorgo_sim_t *sim, uint64_t *n_requests, uint64_t *n_block_ids,
                     uint64_t *n_distinct);

/* Device bytes gorgo_eval_population needs to keep `resident_candidates` replays in flight at
 * once (a population larger than that is evaluated in waves).  Needs an uploaded trace. */
int gorgo_workspace_bytes(const gorgo_sim_t *sim, uint32_t resident_candidates,
                          uint64_t *bytes_out);

/* Section 2.3 (evaluating candidate weights; objective p95 TTFT, Section 4).  Replays the whole
 * uploaded trace once per candidate from the empty state, timestamps multiplied by `time_scale`
 * (Section 3), and reduces each candidate's TTFT and E2E to p95.
 *   params        P*K doubles row-major, HOST or DEVICE (detected); all finite (host copies are
 *                 checked: GORGO_ERR_NONFINITE_PARAM)
 *   workspace     DEVICE scratch of workspace_bytes >= gorgo_workspace_bytes(sim, 1)
 *   p95_ttft_ms,  DEVICE, P doubles each
 *   p95_e2e_ms
 *   route         DEVICE P*N bytes or NULL: chosen replica per candidate and request
 *   hit_blocks    DEVICE P*N uint16 or NULL: prefix-hit length on the chosen replica
 *   state_digest  DEVICE P*R*2 uint64 or NULL: per replica (occupancy, sum over cached blocks of
 *                 mix64(id ^ mix64(seq*65536+pos)) mod 2^64), mix64 = splitmix64 finaliser,
 *                 id = the caller's 64-bit block id, (seq, pos) = request and position of the
 *                 block's last touch
 *   stats         DEVICE P*4 uint64 or NULL: per candidate the sums over requests of
 *                 sum_i min(h_i+1, n), h on the chosen replica, n, evicted blocks
 *   cand_status   DEVICE P int32 or NULL: 0, or nonzero if a bounded loop hit its limit
 * Outputs are valid once `cuda_stream` has been synchronised. */
int gorgo_eval_population(gorgo_sim_t *sim, uint32_t n_candidates, const double *params,
                          double time_scale, void *workspace, uint64_t workspace_bytes,
                          void *cuda_stream, double *p95_ttft_ms, double *p95_e2e_ms,
                          uint8_t *route, uint16_t *hit_blocks, uint64_t *state_digest,
                          uint64_t *stats, int32_t *cand_status);

/* Same evaluation with HOST inputs and outputs: copies `params` (HOST, P*K) to the device,
 * runs, copies p95_ttft_ms / p95_e2e_ms (HOST, P doubles each; pinned memory makes the copies
 * asynchronous) back and waits for the stream.  Returns GORGO_ERR_DEVICE_LIMIT if any candidate
 * reported a nonzero status. */
int gorgo_eval_population_host(gorgo_sim_t *sim, uint32_t n_candidates, const double *params,
                               double time_scale, void *workspace, uint64_t workspace_bytes,
                               void *cuda_stream, double *p95_ttft_ms, double *p95_e2e_ms);

/* Online use (Section 2.3, the proxy routing live requests): one persistent simulator state in
 * caller memory.  gorgo_state_bytes gives its size; gorgo_sim_reset empties it. */
int gorgo_state_bytes(const gorgo_sim_t *sim, uint64_t *bytes_out);
int gorgo_sim_reset(gorgo_sim_t *sim, void *state_workspace, uint64_t state_bytes,
                    void *cuda_stream);

/* Routes requests [first, first+count) of the uploaded trace, in order, with one parameter
 * vector (HOST, K doubles), commits cache and queue state into `state_workspace` (DEVICE) and
 * returns the decisions.  `first` must equal the number of requests the state has already seen
 * (else the state is left untouched and gorgo_state_status reports GORGO_ERR_OUT_OF_ORDER).
 *   route (DEVICE, count bytes), hit_blocks (DEVICE, count uint16, or NULL),
 *   ttft_ms / e2e_ms (DEVICE, count doubles, or NULL). */
int gorgo_route_batch(gorgo_sim_t *sim, const double *params, double time_scale, uint64_t first,
                      uint64_t count, void *state_workspace, uint64_t state_bytes,
                      void *cuda_stream, uint8_t *route, uint16_t *hit_blocks, double *ttft_ms,
                      double *e2e_ms);

/* Digest of the caches held in a persistent state (same definition as state_digest above):
 * `digest` DEVICE R*2 uint64. */
int gorgo_state_digest(gorgo_sim_t *sim, void *state_workspace, uint64_t state_bytes,
                       void *cuda_stream, uint64_t *digest);

/* Waits for `cuda_stream`, then reports how many requests the state has seen and whether a
 * device-side limit or an out-of-order batch was recorded (return value). */
int gorgo_state_status(gorgo_sim_t *sim, void *state_workspace, uint64_t state_bytes,
                       void *cuda_stream, uint64_t *requests_seen);

/* Heterogeneous replicas (the paper's Section 7 names a uniform fleet as a limitation of its
 * cost model): per-replica service speeds for every later replay of this simulator.
 * `prefill_ms_per_token` and `tpot_ms` are HOST arrays of R doubles, finite and >= 0, copied by
 * the call; NULL restores the uniform constant of the configuration for that quantity.  Only the
 * service model uses them (first-token time = start + prefill_i * uncached tokens, finish =
 * first + tpot_i * max(out - 1, 0) on the chosen replica i); the score of Eq. 3 does not see
 * them, as the paper's proxy has no such signal.  A persistent state (gorgo_route_batch) should
 * keep one setting from reset to its last batch. */
int gorgo_sim_set_replica_speeds(gorgo_sim_t *sim, const double *prefill_ms_per_token,
                                 const double *tpot_ms);

/* Proxy index that drifts from the replica's cache (paper Section 7 names it as a limitation: the
 * proxy's prefix index is built from the requests it dispatched and does not observe what the
 * replica evicts).  With `enable` nonzero the score of Eq. 3 takes its prefix hits from the
 * proxy's index of a replica -- every block of every request dispatched to it so far, never
 * forgotten -- while the prefill time, the reported hit length, the cache contents and their
 * digests follow the replica's real LRU cache.  As long as nothing is evicted both are the same.
 * Applies to every later replay of this simulator; a persistent state should keep one setting
 * from reset to its last batch. */
int gorgo_sim_set_proxy_index(gorgo_sim_t *sim, int enable);

/* Time-varying network (paper Section 2.2: the proxy's network signal is an exponentially
 * weighted moving average of an RTT probe sent every 30 s; its Section 4 shows the probes of one
 * run).  `samples_ms` HOST [n_epochs][G][R]: the probe result of every epoch of `epoch_ms`
 * milliseconds of (scaled) trace time, finite and >= 0.  A request that arrives at scaled time t
 * belongs to epoch e = the largest k <= n_epochs-1 with k*epoch_ms <= t.  The score of Eq. 3 uses
 * the proxy's signal of that epoch, ewma_0 = sample_0, ewma_e = ewma_{e-1} + alpha*(sample_e -
 * ewma_{e-1}) (0 < alpha <= 1, three rounded operations, computed by this call); the delay the
 * request experiences on its way to the engine is the epoch's probe itself.  A constant series
 * gives bit-identical results to the static matrix of the configuration.  n_epochs = 0 restores
 * the static matrix.  The series is copied; it applies to every later replay of this simulator
 * (gorgo_workspace_bytes and gorgo_state_bytes grow by 16*n_epochs*G*R bytes: call them again). */
int gorgo_sim_set_rtt_series(gorgo_sim_t *sim, uint32_t n_epochs, double epoch_ms, double alpha,
                             const double *samples_ms);

/* Extended service model (the paper's Section 2.2 describes continuous batching as "bounded by
 * max concurrency and KV budget"; its Section 5 and Appendix D report that concentrating traffic
 * on one replica lowers TTFT but inflates end-to-end latency).  Both parts are this library's
 * statement, off by default, and apply to every later replay of this simulator:
 *   decode_slowdown g >= 0   a request's time per output token is tpot_i * (1 + g*(b-1)), where
 *                            b counts the replica's slots that are busy at the request's
 *                            first-token time, its own included (fixed at that time: the request
 *                            neither speeds up later nor slows the requests already running);
 *   kv_budget_tokens > 0     a request holds input + output tokens of KV while it runs.  On the
 *                            slot that frees first it starts at the earliest time T >= arrival,
 *                            T >= the slot's free time, at which the newest requests of the other
 *                            slots still busy at T hold at most kv_budget_tokens minus its own
 *                            need (T moves from one finish time of those slots to the next); once
 *                            no other slot is busy it starts whatever its size.  0 = no budget.
 * Only the service model changes (start, first-token and finish times); the score of Eq. 3 does
 * not see it.  With g = 0 and no budget every result is bit-identical to the plain model.  A
 * persistent state should keep one setting from reset to its last batch. */
int gorgo_sim_set_service_model(gorgo_sim_t *sim, double decode_slowdown, uint64_t kv_budget_tokens);

/* Population evaluation with one time scale per candidate (paper Section 3: the time between
 * requests is scaled linearly to move the load; its load sweep replays one trace at several
 * scales).  Candidate p is replayed with time_scales[p]; everything else is
 * gorgo_eval_population.  A sweep of S scales over P parameter vectors is then ONE population of
 * S*P (parameter vector, scale) pairs, which fills the GPU better than S evaluations of P: a
 * replay occupies its share of an SM for the whole trace, so a population slightly larger than
 * the number of replays the GPU holds at once costs two rounds.  `time_scales` HOST, P doubles,
 * finite and >= 0; `params` HOST or DEVICE; outputs DEVICE as for gorgo_eval_population.  The
 * call waits for `cuda_stream`. */
int gorgo_eval_population_scales(gorgo_sim_t *sim, uint32_t n_candidates, const double *params,
                                 const double *time_scales, void *workspace,
                                 uint64_t workspace_bytes, void *cuda_stream, double *p95_ttft_ms,
                                 double *p95_e2e_ms, uint8_t *route, uint16_t *hit_blocks,
                                 uint64_t *state_digest, int32_t *cand_status);

/* Baseline routing policies of the paper (Section 4, "Baseline policies"; `random` is in its
 * appendix tables) replayed through the same simulator, so that their TTFT/E2E can be set beside
 * a tuned cost model's.  The paper runs them against live engines; inside the simulator they read:
 *   LEAST_LOAD        fewest in-flight input tokens recorded by the proxy (the engine-side terms
 *                     of the paper's sum do not exist here): the cost model with weights (0,0,1);
 *   LEAST_REQUEST     fewest in-flight requests: the same with the queue signal counted in
 *                     requests (in flight as for tokens: finish time > arrival);
 *   PREFIX_CACHE      longest cached prefix: weights (0,1,0);
 *   SESSION_AFFINITY  the paper hashes the first 256 tokens of the prompt; the id of the first
 *                     block stands for them: replica = finaliser(id) mod R, with the 64-bit
 *                     finaliser z ^= z>>30; z *= 0xbf58476d1ce4e5b9; z ^= z>>27;
 *                     z *= 0x94d049bb133111eb; z ^= z>>31; replica 0 for a prompt without blocks;
 *   RANDOM            replica = draws[r] mod R; `draws` HOST, one uint32 per request of the trace
 *                     (the caller's random numbers; NULL for the other policies).
 * Ties go to the lowest replica index.  One replay from the empty state; outputs as for
 * gorgo_eval_population with one candidate: `p95_ttft_ms`, `p95_e2e_ms` DEVICE 1 double each,
 * `route` DEVICE N bytes or NULL, `hit_blocks` DEVICE N uint16 or NULL, `state_digest` DEVICE
 * R*2 uint64 or NULL, `cand_status` DEVICE 1 int32 or NULL.  `workspace` as for
 * gorgo_eval_population with one resident candidate.  The call waits for `cuda_stream`. */
enum {
  GORGO_POLICY_LEAST_LOAD = 0,
  GORGO_POLICY_LEAST_REQUEST = 1,
  GORGO_POLICY_PREFIX_CACHE = 2,
  GORGO_POLICY_SESSION_AFFINITY = 3,
  GORGO_POLICY_RANDOM = 4
};
int gorgo_eval_policy(gorgo_sim_t *sim, uint32_t policy, const uint32_t *draws, double time_scale,
                      void *workspace, uint64_t workspace_bytes, void *cuda_stream,
                      double *p95_ttft_ms, double *p95_e2e_ms, uint8_t *route,
                      uint16_t *hit_blocks, uint64_t *state_digest, int32_t *cand_status);

/* Rolling-window tuning objective (paper Section 4: the online tuner minimises the p95 TTFT of
 * a rolling 128-request window with hop 32; the caption of its convergence figure reports the
 * best window).  Window j covers requests [j*hop, j*hop + window) in trace order and its value is
 * the nearest-rank p95 of their TTFTs, the k-th smallest with k = ceil(0.95 * window);
 * n_windows = (N - window) / hop + 1 (gorgo_window_count), 0 when N < window.
 * gorgo_eval_population_windows replays the population like gorgo_eval_population and reduces
 * each candidate's TTFTs to: `win_p95_ttft_ms` DEVICE P*n_windows doubles, row-major, or NULL;
 * `best_win_p95_ttft_ms` DEVICE P doubles, the smallest window value (required);
 * `best_window` DEVICE P uint32, the first window that attains it, or NULL; `p95_ttft_ms` and
 * `p95_e2e_ms` DEVICE P doubles each, the whole-replay p95s, both or neither NULL;
 * `cand_status` DEVICE P int32 or NULL.  `params` HOST or DEVICE.  Work is enqueued on
 * `cuda_stream`.  Errors: GORGO_ERR_INVALID_ARG for window = 0, hop = 0, window > 2048 or
 * N < window; otherwise those of gorgo_eval_population. */
int gorgo_window_count(uint64_t n_requests, uint32_t window, uint32_t hop, uint64_t *n_windows);
int gorgo_eval_population_windows(gorgo_sim_t *sim, uint32_t n_candidates, const double *params,
                                  double time_scale, void *workspace, uint64_t workspace_bytes,
                                  void *cuda_stream, uint32_t window, uint32_t hop,
                                  double *win_p95_ttft_ms, double *best_win_p95_ttft_ms,
                                  uint32_t *best_window, double *p95_ttft_ms, double *p95_e2e_ms,
                                  int32_t *cand_status);

/* Evolution strategy of the tuner (paper Section 2.3: a (1+1)-ES perturbs each tuned weight
 * multiplicatively in log space, Eq. 4  x' = clip(exp(ln x + sigma z), [lo, hi]), keeps the
 * offspring when it beats the parent on the objective, and adapts sigma by Rechenberg's 1/5
 * success rule; Section 4: W_rtt and W_queue start at 0.5 and 0.1 in [0.05, 2.0] and
 * [0.05, 0.5], sigma0 = 0.5).  Here the strategy runs offline on the batched evaluator: step t
 * draws `lambda` offspring of the parent (lambda = 1 is the paper's strategy), replays them over
 * the uploaded trace in one population evaluation, takes the one with the smallest objective
 * (lowest index among equals) and accepts it iff its objective is strictly smaller than the
 * parent's.  The paper leaves the constants of the 1/5 rule open: sigma is multiplied by
 * `sigma_up` after an accepted step and by sigma_up^(-1/4) after a rejected one, which leaves it
 * unchanged at exactly one success in five.  The normal draws are an input: z[(t*lambda + l)*
 * n_tuned + k] perturbs tuned parameter k of offspring l in step t.  Parameters not listed in
 * `tuned` keep their value from x0.  The arithmetic of Eq. 4 is done on the host in double
 * precision with the C library's exp and log; the sum ln x + sigma*z is two rounded operations.
 * All pointers are HOST except `workspace` (DEVICE, as for gorgo_eval_population).  The call
 * synchronises `cuda_stream` once per step.  `history`, if not NULL, receives per step
 * 4 + n_tuned doubles: objective of the best offspring, 1.0 if it was accepted else 0.0, sigma
 * after the step, objective of the parent after the step, tuned values of the parent after the
 * step.  Errors: GORGO_ERR_INVALID_ARG (NULL, lambda = 0, n_tuned = 0 or > K, an index >= K,
 * lo <= 0, hi < lo, x0 of a tuned parameter <= 0, objective > 1), GORGO_ERR_NONFINITE_PARAM,
 * and those of gorgo_eval_population. */
typedef struct {
  uint32_t n_steps;        /* ES steps                                                       */
  uint32_t lambda;         /* offspring per step                                             */
  uint32_t n_tuned;        /* number of tuned parameters                                     */
  uint32_t objective;      /* 0: p95 TTFT of the replay (the paper's), 1: p95 E2E            */
  const uint32_t *tuned;   /* [n_tuned] their indices in the K-vector                        */
  const double *lo;        /* [n_tuned] lower clamp, > 0                                     */
  const double *hi;        /* [n_tuned] upper clamp, >= lo                                   */
  double sigma0;           /* initial step size, > 0                                         */
  double sigma_up;         /* > 1                                                            */
  double time_scale;       /* as for gorgo_eval_population                                   */
} gorgo_es_config_t;
int gorgo_es_run(gorgo_sim_t *sim, const gorgo_es_config_t *cfg, const double *x0,
                 const double *z, void *workspace, uint64_t workspace_bytes, void *cuda_stream,
                 double *x_best, double *objective_best, double *sigma_final, double *history);

/* The paper's tuner as it runs in the proxy (Section 2.3; Section 4): ONLINE, inside one replay.
 * The weights in force change every `hop` requests.  Step k = 1, 2, ... of the (1+1)-ES takes
 * place when window + (k-1)*hop requests have been routed (window 128, hop 32: the 18th step
 * after 672 samples, as the paper counts) and is scored by the nearest-rank p95 of the TTFTs of
 * the last `window` requests in trace order.  Step 1 scores the start weights.  Every later step
 * scores the offspring that was in force during the last hop (the window still holds requests
 * routed under earlier weights, as a rolling window does), makes it the parent iff its value is
 * strictly smaller than the parent's, multiplies sigma by `sigma_up` after an accepted step and
 * by sigma_up^(-1/4) after a rejected one, and puts a new offspring of the parent (Eq. 4, clamped to
 * [lo, hi]) in force for the next hop.  After `n_draw_steps` steps the weights in force stay.
 * `n_tuners` independent tuners run side by side, each on its own simulator state, from its own
 * start weights and draws: x0 HOST [n_tuners*K]; z HOST [n_tuners * n_draw_steps * n_tuned],
 * z[(p*n_draw_steps + (k-1))*n_tuned + j] perturbs tuned parameter j of tuner p in step k.
 * The replays, the window values and the final p95s are computed on the device; Eq. 4 and the
 * accept/reject bookkeeping run on the host between the chunks (C library exp and log, the sum
 * ln x + sigma*z two rounded operations), so the call synchronises `cuda_stream` once per hop.
 * Outputs (HOST unless noted): x_final [n_tuners*K] the parents at the end; sigma_final
 * [n_tuners]; steps_done (may be NULL) the steps taken, min(n_draw_steps, number of full windows);
 * history, or NULL, [n_tuners * n_draw_steps * (4 + 2*n_tuned)]: per tuner and step the window
 * value, 1.0 if accepted else 0.0, sigma after the step, the parent's value after the step, the
 * parent's tuned weights after the step, the tuned weights put in force for the next hop;
 * p95_ttft_ms / p95_e2e_ms [n_tuners] each, both or neither NULL: p95 over the whole tuned replay;
 * route DEVICE [n_tuners*N] bytes or NULL.  `workspace` DEVICE, at least
 * gorgo_workspace_bytes(sim, n_tuners): all tuners stay resident.  Errors: those of gorgo_es_run;
 * GORGO_ERR_WORKSPACE_TOO_SMALL if the tuners do not all fit. */
typedef struct {
  uint32_t n_tuned;        /* number of tuned parameters                                     */
  uint32_t n_draw_steps;   /* steps for which z holds draws                                  */
  uint32_t window, hop;    /* rolling window and hop in requests (paper: 128, 32); window <= 2048 */
  const uint32_t *tuned;   /* [n_tuned] their indices in the K-vector                        */
  const double *lo;        /* [n_tuned] lower clamp, > 0                                     */
  const double *hi;        /* [n_tuned] upper clamp, >= lo                                   */
  double sigma0;           /* initial step size, > 0                                         */
  double sigma_up;         /* > 1                                                            */
  double time_scale;       /* as for gorgo_eval_population                                   */
} gorgo_online_config_t;
int gorgo_tune_online(gorgo_sim_t *sim, const gorgo_online_config_t *cfg, uint32_t n_tuners,
                      const double *x0, const double *z, void *workspace, uint64_t workspace_bytes,
                      void *cuda_stream, double *x_final, double *sigma_final, uint32_t *steps_done,
                      double *history, double *p95_ttft_ms, double *p95_e2e_ms, uint8_t *route);

/* Measurement aid (no counterpart in the paper): how many candidates (CTAs of the replay kernel)
 * one SM holds at once for this configuration, and the shared memory each takes.  A population
 * larger than SMs x that number is replayed in successive rounds of CTAs. */
int gorgo_replay_occupancy(gorgo_sim_t *sim, int32_t *ctas_per_sm, uint64_t *smem_bytes_per_cta);
/* Measurement aid (no counterpart in the paper).  With profiling enabled, gorgo_eval_population
 * records a CUDA event on `cuda_stream` directly before and after each launch of the replay
 * kernel (one launch per wave, at most 32 waves are timed).  gorgo_last_replay_ms waits for those
 * events and returns the summed device time of the replay launches of the most recent
 * evaluation and their number. */
int gorgo_set_profiling(gorgo_sim_t *sim, int enable);
int gorgo_last_replay_ms(gorgo_sim_t *sim, double *replay_ms, uint32_t *launches);
/* The same for the window-objective kernels of the most recent gorgo_eval_population_windows. */
int gorgo_last_window_ms(gorgo_sim_t *sim, double *window_ms, uint32_t *launches);

/* Measurement aid (no counterpart in the paper): the rate at which this GPU serves independent
 * 32-byte reads (one sector each) at pseudo-random positions of a footprint of `footprint_bytes`,
 * in GB/s of sectors (reads x 32 bytes / time; best of three timed launches after a warm-up, CUDA
 * events on `cuda_stream`).  With a footprint far larger than the L2 cache this is the random-sector
 * DRAM rate, with a footprint inside it the L2 rate: the two yardsticks a gather-bound kernel can be
 * held against besides the streaming copy bandwidth.  `buffer` DEVICE, 256-byte aligned,
 * `buffer_bytes` >= footprint_bytes + 256 (its contents are read, and four bytes behind the
 * footprint may be written); footprint_bytes >= 4096.  The call waits for its launches. */
int gorgo_measure_gather(int device, void *buffer, uint64_t buffer_bytes, uint64_t footprint_bytes,
                         void *cuda_stream, double *sectors_gb_per_s);

/* Test aid (no counterpart in the paper).  Inside the replay kernel the warps of one candidate
 * wait for one another with bounded polls, and two kinds of helper warps only prepare work
 * ahead of the warps that must do it anyway (the probe warps stage prefix hits, the scout warps
 * pre-validate eviction victims).  These switches let a test take those paths on purpose; none
 * of them makes a kernel fault or hang.  They apply to every later launch of `sim`.
 *   GORGO_DEBUG_POLL_LIMIT  polls after which a warp gives up waiting (default 2^24).  With 0 the
 *                           first wait that is not already satisfied gives up: the candidate
 *                           finishes with wrong results and status GORGO_ERR_DEVICE_LIMIT.
 *   GORGO_DEBUG_RING_POLLS  polls of a commit warp for the scout's next victim before it looks for
 *                           victims itself (default 64; results do not depend on it).
 *   GORGO_DEBUG_PROBE_OFF   nonzero: no probe warps; every request is probed where it is needed
 *                           (results do not depend on it).
 *   GORGO_DEBUG_SCOUT_OFF   nonzero: no scout warps (results do not depend on it). */
enum {
  GORGO_DEBUG_POLL_LIMIT = 0,
  GORGO_DEBUG_RING_POLLS = 1,
  GORGO_DEBUG_PROBE_OFF = 2,
  GORGO_DEBUG_SCOUT_OFF = 3
};
int gorgo_debug_set(gorgo_sim_t *sim, uint32_t what, uint32_t value);

/* Population evaluation for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a packaging variant of gorgo_eval_population).  Some hosts of this library
 * own no allocator they may call at the moment they want a score: code running inside another
 * framework's memory plan whose pool is already carved up, a plugin that was handed its input
 * and output buffers and nothing else, a latency-critical control loop (the proxy re-tuning its
 * weights) that must not hit cudaMalloc's implicit device synchronisation.  For them the replay
 * scratch (cache masks, replica and slot state, per-request chains, latency arrays) lives in an
 * array compiled into the library, GORGO_STATIC_SCRATCH_BYTES long, that every GPU which loads
 * the library holds until the process exits.  The call allocates and frees nothing, on host
 * paths of the CUDA runtime included: no cudaMalloc, cudaFree or allocating library routine.
 *
 * Arguments are those of gorgo_eval_population without the workspace, digest and counters:
 * `params` HOST or DEVICE (P*K doubles), `p95_ttft_ms` / `p95_e2e_ms` DEVICE (P doubles
 * each), `route` DEVICE P*N bytes or NULL, `hit_blocks` DEVICE P*N uint16 or NULL, `cand_status`
 * DEVICE P int32 or NULL: 0, or GORGO_ERR_DEVICE_LIMIT for a candidate whose replay gave up on a
 * bounded wait (its outputs are then meaningless; read it after synchronising the stream).
 * Limit: the scratch of ONE candidate, gorgo_workspace_bytes(sim, 1), must not exceed
 * GORGO_STATIC_SCRATCH_BYTES, else GORGO_ERR_STATIC_LIMIT and nothing runs; a population whose
 * candidates do not all fit at once is evaluated in waves.  (Per candidate the scratch is about
 * 41 bytes per request plus 1 to 8 bytes per distinct block id.)
 * The first call on a device looks up the array's device address; make that first call outside
 * any stream capture.  All calls in a process share the one array per GPU and it keeps what the
 * previous call left there; each call clears what it needs to start from zero, but two calls
 * whose GPU work overlaps (different streams, different handles, different threads) race on it:
 * serialise them. */
#define GORGO_STATIC_SCRATCH_BYTES (64u << 20)
int gorgo_eval_population_static(gorgo_sim_t *sim, uint32_t n_candidates, const double *params,
                                 double time_scale, void *cuda_stream, double *p95_ttft_ms,
                                 double *p95_e2e_ms, uint8_t *route, uint16_t *hit_blocks,
                                 int32_t *cand_status);

const char *gorgo_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* GORGO_H_ */

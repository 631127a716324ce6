// Internal declarations shared by the host shell and the kernels of libgorgo_b200.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gorgo {

constexpr uint32_t kNone = 0xFFFFFFFFu;

// One request of the trace as the kernels read it: exactly one 32-byte sector.
struct __align__(32) ReqRec {
  double ts_ms;       // arrival at the proxy (unscaled)
  uint32_t off;       // first block id of the request in the flat id array
  uint32_t in_tok;    // input tokens
  uint32_t out_tok;   // output tokens
  uint16_t nblk;      // number of blocks
  uint16_t origin;    // origin region
  uint32_t prev_share;  // latest earlier request that shares a block with this one (kNone: none)
  uint32_t pad;
};
static_assert(sizeof(ReqRec) == 32, "ReqRec must be one sector");

// Per-(candidate, replica) scalars kept in global memory between launches.
struct __align__(32) RepState {
  long long load;     // in-flight input tokens
  long long cnt;      // in-flight requests
  uint32_t occ;       // cached blocks
  uint32_t cur_req;   // eviction cursor: request whose touches are examined next (kNone: none yet)
  int32_t cur_pos;    //   next position of that request to examine (counts down; <0: exhausted)
  uint32_t lru_tail;  // last request routed to this replica (kNone: none yet)
};
static_assert(sizeof(RepState) == 32, "RepState layout");

// Header of one candidate's state block.
struct __align__(32) CandHeader {
  uint32_t processed;  // requests replayed so far
  int32_t status;      // 0, or a gorgo_status recorded by a kernel
  uint32_t overflow;   // persistent state: 1 + the newest request that completes after the end of
                       // the trace known so far (0: none); such requests are chained through
                       // their completion records until an appended request takes them
  uint32_t pad[5];
};

// Device-resident trace (pointers into the caller's trace buffer).
struct TraceView {
  const ReqRec* req;       // [N]
  const uint32_t* ids;     // [T] dense block ids, request after request
  const uint2* occ_next;   // [T] (.x = flat index of the next occurrence of the same block or
                           //      kNone, .y = request of that occurrence)
  const uint2* occ_prev;   // [T] the same for the previous occurrence
  const uint64_t* raw_id;  // [D] caller's 64-bit id of each dense id
  const double* ts;        // [N] arrival times (unscaled), the same values as in `req`
  // time grid over the unscaled arrival times: grid[b] = first request with ts >= b * grid_dt,
  // b = 0..grid_n (grid_n = 0: no grid, e.g. all arrivals at one instant)
  const uint32_t* grid;
  double grid_dt;
  uint32_t grid_n;
  uint32_t n_req, n_ids, n_distinct;
};

// Model constants.
struct Model {
  uint32_t R, G, S, B, K;
  uint64_t C;
  double prefill_ms, tpot_ms;
};

// Layout of one candidate's state block (bytes from its start); the mask array of the
// candidate lives in a separate region.
struct StateLayout {
  uint64_t rep_off;        // RepState[R]
  uint64_t slot_off;       // double[R*S]: time each slot frees (finish of its newest request)
  uint64_t slot_kv_off;    // uint64[R*S]: KV tokens held by each slot's newest request
  uint64_t bytes;          // size of the block (multiple of 256)
};

// Everything one replay launch needs.  Candidate p of the launch uses element/byte strides.
struct ReplayArgs {
  Model m;
  TraceView tr;
  double scale;
  const double* scales;           // [P] device, one time scale per candidate, or null (use `scale`)
  uint32_t first, count;          // requests [first, first+count)
  uint32_t check_order;           // 1: refuse (status) unless header.processed == first
  uint32_t poll_limit;            // polls after which a warp stops waiting for another one
  uint32_t ring_polls;            // polls of a commit warp for the scout's next victims before it walks itself
  uint32_t probe_off, scout_off;  // test switches: run without the probe warp / without the scout warps
  uint32_t slots_in_smem;         // set by the launcher: per-slot state fits in shared memory
  uint32_t lists_in_smem;         // set by the launcher: eviction lists fit in shared memory
  uint4* evict_lists;             // [P * evict_list_bytes(R)] scratch used when they do not
  const double* rtt;              // [G*R] device
  const double* params;           // [P*K] device
  unsigned char* masks;           // [P * mask_stride] bytes
  uint64_t mask_stride;           // bytes per candidate
  unsigned char* states;          // [P * layout.bytes]
  StateLayout lay;
  // per-request arrays, candidate p at + p*N elements
  uint32_t* exp_head;             // [r]: first entry of the list of requests whose completion the
                                  //   proxy sees when request r arrives (kNone: none)
  uint4* exp_rec;                 // [j]: (next entry of j's list, input tokens of j, replica of j, -)
  uint32_t* lru_next;             // next request routed to the same replica
  uint8_t* route_log;             // chosen replica of every request replayed so far
  uint64_t route_log_stride;      // elements between candidates
  // baseline policies: queue signal counted in requests instead of tokens; one fixed route per
  // request of the trace (shared by the candidates of the launch) or null
  uint32_t queue_in_requests;
  const uint8_t* forced_route;
  // heterogeneous replicas: per-replica prefill ms per token and ms per output token (device
  // [R] each) or null for the uniform constants of the model
  const double* rep_prefill_ms;
  const double* rep_tpot_ms;
  // persistent state only: finish time of every request that completes after the trace's end
  double* finish_log;
  // 1: the score takes prefix hits from the proxy's own index (blocks ever dispatched to a
  // replica) instead of the replica's cache
  uint32_t proxy_index;
  // time-varying network: per epoch the proxy's RTT signal (EWMA of the probes) and the probes
  // themselves (the delay a request experiences), [n_epochs][G][R] each, device; null = static
  const double* rtt_ewma;
  const double* rtt_raw;
  uint32_t n_epochs;
  double epoch_ms;
  // extended service model (0 = off): decode slow-down per additional busy slot, KV budget of a
  // replica in tokens
  double decode_slowdown;
  unsigned long long kv_budget;
  // outputs, candidate p at + p*out_stride, request r at + (r-first); any may be null
  uint8_t* route_out;
  uint16_t* hit_out;
  double* ttft_out;
  double* e2e_out;
  uint64_t out_stride;
  uint64_t* stats;                // [P*4] or null (accumulated)
  int32_t* status_out;            // [P] or null
};

struct SelectArgs {
  const double* ttft;             // [P*stride]
  const double* e2e;
  uint64_t stride;
  uint32_t n;                     // values per candidate
  double* p95_ttft;               // [P]
  double* p95_e2e;
};

struct WindowArgs {
  const double* values;           // [P*stride] per-request values (TTFT), request order
  uint64_t stride;
  uint32_t window, hop, n_win;    // window j covers values [j*hop, j*hop + window)
  double* win_p95;                // [P*win_stride] window values (output, also input of the best)
  uint64_t win_stride;
  double* best;                   // [P] smallest window value
  uint32_t* best_win;             // [P] first window attaining it, or null
};

struct DigestArgs {
  Model m;
  TraceView tr;
  const unsigned char* states;
  StateLayout lay;
  const uint8_t* route_log;
  uint64_t route_log_stride;
  uint64_t* digest;               // [P*R*2], zeroed by the launcher
};

cudaError_t launch_reset(unsigned char* masks, uint64_t mask_bytes_total, uint32_t* exp_head,
                         uint64_t exp_head_count, unsigned char* states, const StateLayout& lay,
                         const Model& m, uint32_t n_cand, cudaStream_t st);
cudaError_t launch_replay(const ReplayArgs& a, uint32_t n_cand, cudaStream_t st);
cudaError_t launch_select(const SelectArgs& a, uint32_t n_cand, cudaStream_t st);
cudaError_t launch_digest(const DigestArgs& a, uint32_t n_cand, cudaStream_t st);
cudaError_t launch_window(const WindowArgs& a, uint32_t n_cand, cudaStream_t st);
cudaError_t launch_policy_routes(const TraceView& tr, uint32_t R, bool affinity,
                                 const uint32_t* draws, uint8_t* route, cudaStream_t st);
#ifdef GORGO_PROF
// Cycle accounting build only: the 64 accumulators (route warp at 0, service at 16, gate at 32, commit warps at 48).
cudaError_t prof_read(unsigned long long* out64, bool reset);
#endif
// After requests [first_new, first_new + n_new) were appended: every block of theirs whose previous
// occurrence lies before flat position `ids_before` becomes that occurrence's successor.
cudaError_t launch_link_occurrences(const TraceView& tr, uint32_t first_new, uint32_t n_new,
                                    uint32_t ids_before, uint2* occ_next, cudaStream_t st);
cudaError_t launch_gather(const void* buf, uint64_t n_sectors, uint32_t per_thread, uint32_t blocks,
                          uint32_t* sink, cudaStream_t st);
uint32_t window_max();          // largest window the window kernel handles
uint32_t mask_bytes_for(uint32_t n_replicas);
uint64_t evict_list_bytes(uint32_t n_replicas);
// CTAs of the replay kernel that fit one SM for this model (-1: query failed), and the dynamic
// shared memory one CTA asks for.
int replay_occupancy(const Model& m, uint64_t* smem_bytes);

}  // namespace gorgo

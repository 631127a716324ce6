// Host shell of libgorgo_b200: the C ABI declared in include/gorgo.h.  Argument checks, trace
// preparation (validation, dense renumbering of block ids, next-occurrence links), workspace
// layout, wave scheduling and kernel launches.  No step of the simulation runs on the host.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <memory>
#include <vector>

#include "../../include/gorgo.h"
#include "gorgo_internal.h"

using namespace gorgo;

// 64-bit id -> dense number, open addressing, grows by doubling.
struct IdMap {
  std::vector<uint64_t> keys;
  std::vector<uint32_t> vals;  // 0 = empty, else dense + 1
  uint64_t mask = 0, used = 0;
  static uint64_t hash(uint64_t z) {
    z ^= z >> 33; z *= 0xff51afd7ed558ccdULL; z ^= z >> 33; z *= 0xc4ceb9fe1a85ec53ULL;
    return z ^ (z >> 33);
  }
  explicit IdMap(uint64_t cap_pow2) : keys(cap_pow2), vals(cap_pow2, 0), mask(cap_pow2 - 1) {}
  void grow() {
    IdMap bigger((mask + 1) * 2);
    for (uint64_t i = 0; i <= mask; ++i)
      if (vals[i]) bigger.put(keys[i], vals[i]);
    keys.swap(bigger.keys); vals.swap(bigger.vals); mask = bigger.mask;
  }
  void put(uint64_t k, uint32_t v) {
    uint64_t i = hash(k) & mask;
    while (vals[i]) i = (i + 1) & mask;
    keys[i] = k; vals[i] = v; ++used;
  }
  // returns dense number, assigning `next` if the id is new
  uint32_t get_or_add(uint64_t k, uint32_t& next) {
    uint64_t i = hash(k) & mask;
    while (vals[i]) {
      if (keys[i] == k) return vals[i] - 1;
      i = (i + 1) & mask;
    }
    if ((used + 1) * 2 > mask + 1) { grow(); return get_or_add(k, next); }
    keys[i] = k; vals[i] = next + 1; ++used;
    return next++;
  }
};

// Host side of a trace that is still growing (gorgo_trace_begin / gorgo_trace_append): what the
// next batch needs to know about the requests before it, and where the device regions lie.
struct TraceBuilder {
  IdMap map{1ull << 16};
  std::vector<uint32_t> seen_in;          // per dense id: request (+1) that last contained it
  std::vector<uint32_t> last_g, last_r;   // per dense id: flat position and request of its last occurrence
  std::vector<uint64_t> raw_new;          // caller's ids of the dense ids added by the current batch
  std::vector<double> ts;                 // arrival times so far
  uint64_t cap_req = 0, cap_ids = 0;      // capacities the device regions were laid out for
  uint64_t N = 0, T = 0;
  uint32_t D = 0;
  double grid_dt = 0.0;
  uint32_t grid_n = 0;
  uint64_t grid_cursor = 0;               // first request not yet behind the last grid edge
  unsigned char *d_req = nullptr, *d_ids = nullptr, *d_occ = nullptr, *d_raw = nullptr,
                *d_prev = nullptr, *d_ts = nullptr, *d_grid = nullptr;
};

struct gorgo_sim {
  Model m;
  std::unique_ptr<TraceBuilder> tb;       // set while the trace can still grow
  uint64_t cap_req = 0, cap_ids = 0;      // appendable trace: sizes the workspaces are laid out for (else 0)
  std::vector<double> rtt;
  std::vector<double> rep_prefill, rep_tpot;   // per-replica speeds; empty: the uniform constants
  double decode_slowdown = 0.0;                // extended service model (0: off)
  uint64_t kv_budget = 0;
  uint32_t proxy_index = 0;                    // score with the proxy's own index instead of the cache
  std::vector<double> rtt_raw, rtt_ewma;       // time-varying network, [n_epochs][G][R] each; empty: static
  uint32_t n_epochs = 0;
  double epoch_ms = 0.0;
  int device = 0;
  bool has_trace = false;
  TraceView tr = {};
  uint32_t poll_limit = 1u << 24;   // bound of the device-side waits of one warp for another
  uint32_t ring_polls = 64;         // polls for the scout's victims before a commit warp walks itself
  uint32_t probe_off = 0, scout_off = 0;   // test switches (gorgo_debug_set)
  // optional CUDA-event timing of the replay kernel (one pair per wave of the last evaluation)
  bool profiling = false;
  std::vector<cudaEvent_t> ev;    // pairs around the replay launches
  uint32_t ev_used = 0;
  std::vector<cudaEvent_t> wev;   // pairs around the window-objective launches
  uint32_t wev_used = 0;
};

namespace {

constexpr uint64_t kAlign = 256;
inline uint64_t align_up(uint64_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

StateLayout make_layout(const Model& m) {
  StateLayout l;
  uint64_t o = sizeof(CandHeader);
  l.rep_off = o; o += (uint64_t)m.R * sizeof(RepState);
  const uint64_t rs = (uint64_t)m.R * m.S;
  l.slot_off = o; o += rs * 8;
  l.slot_kv_off = o; o += rs * 8;
  l.bytes = align_up(o);
  return l;
}

// Byte offsets of the regions of a workspace for `res` resident candidates.
struct WsLayout {
  uint64_t params, scales, rtt, speeds, status, p95, forced, draws, series, masks, states, lists, exp_head, exp_rec, lru_next,
      route_log, finish, ttft, e2e, total;
  uint64_t mask_stride;
  StateLayout st;
};

WsLayout make_ws(const gorgo_sim* s, uint64_t res, bool with_latency) {
  WsLayout w;
  const Model& m = s->m;
  // an appendable trace lays everything out for its capacities, so that a persistent state stays
  // valid while the trace grows
  const uint64_t N = s->cap_req ? s->cap_req : s->tr.n_req;
  const uint64_t D = s->cap_req ? s->cap_ids : s->tr.n_distinct;
  w.st = make_layout(m);
  w.mask_stride = align_up(D * mask_bytes_for(m.R));
  uint64_t o = 0;
  w.params = o; o = align_up(o + res * m.K * 8);
  w.scales = o; o = align_up(o + res * 8);       // one time scale per candidate (optional)
  w.rtt = o; o = align_up(o + (uint64_t)m.G * m.R * 8);
  w.speeds = o; o = align_up(o + (uint64_t)m.R * 16);   // per-replica speeds (optional)
  w.series = o; o = align_up(o + (uint64_t)s->n_epochs * m.G * m.R * 16);   // RTT series (optional)
  w.status = o; o = align_up(o + res * 4);
  w.p95 = o; o = align_up(o + res * 16);
  w.forced = o; o = align_up(o + N);          // baseline policies: one route per request
  w.draws = o; o = align_up(o + N * 4);       //   and the caller's draws for `random`
  w.masks = o; o = align_up(o + res * w.mask_stride);
  w.states = o; o = align_up(o + res * w.st.bytes);
  w.lists = o; o = align_up(o + res * evict_list_bytes(m.R));
  w.exp_head = o; o = align_up(o + res * N * 4);
  w.exp_rec = o; o = align_up(o + res * N * 16);
  w.lru_next = o; o = align_up(o + res * N * 4);
  w.route_log = o; o = align_up(o + res * N);
  w.finish = o; if (!with_latency) o = align_up(o + res * N * 8);   // persistent state only
  w.ttft = o; if (with_latency) o = align_up(o + res * N * 8);
  w.e2e = o; if (with_latency) o = align_up(o + res * N * 8);
  w.total = o;
  return w;
}

// Copies the per-replica speeds (if set) into the workspace and points the launch at them.
int attach_speeds(const gorgo_sim* sim, unsigned char* base, const WsLayout& w, cudaStream_t st,
                  ReplayArgs* a) {
  const uint32_t R = sim->m.R;
  a->decode_slowdown = sim->decode_slowdown;
  a->kv_budget = sim->kv_budget;
  a->proxy_index = sim->proxy_index;
  if (sim->n_epochs > 0) {
    const size_t n = sim->rtt_raw.size();
    double* ds = reinterpret_cast<double*>(base + w.series);
    if (cudaMemcpyAsync(ds, sim->rtt_ewma.data(), n * 8, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ds + n, sim->rtt_raw.data(), n * 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return GORGO_ERR_CUDA;
    a->rtt_ewma = ds; a->rtt_raw = ds + n;
    a->n_epochs = sim->n_epochs; a->epoch_ms = sim->epoch_ms;
  }
  double* d = reinterpret_cast<double*>(base + w.speeds);
  if (!sim->rep_prefill.empty()) {
    if (cudaMemcpyAsync(d, sim->rep_prefill.data(), R * 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return GORGO_ERR_CUDA;
    a->rep_prefill_ms = d;
  }
  if (!sim->rep_tpot.empty()) {
    if (cudaMemcpyAsync(d + R, sim->rep_tpot.data(), R * 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return GORGO_ERR_CUDA;
    a->rep_tpot_ms = d + R;
  }
  return GORGO_OK;
}

bool is_device_pointer(const void* p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
  return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

bool all_finite(const double* v, uint64_t n) {
  for (uint64_t i = 0; i < n; ++i)
    if (!std::isfinite(v[i])) return false;
  return true;
}

bool finite_nonneg(double v) { return std::isfinite(v) && v >= 0.0; }

// Rolling-window objective asked for with an evaluation (all pointers DEVICE).
// Baseline policy asked for with an evaluation.
struct PolicySpec {
  bool queue_in_requests;
  const uint8_t* forced_route;   // DEVICE [N] or null
};

struct WindowSpec {
  uint32_t window, hop;
  double* win_p95;      // [P * n_windows] or null
  double* best;         // [P]
  uint32_t* best_win;   // [P] or null
};

uint64_t window_count(uint64_t n_requests, uint32_t window, uint32_t hop) {
  return n_requests >= window ? (n_requests - window) / hop + 1 : 0;
}

int eval_impl(gorgo_sim* sim, uint32_t P, const double* params, double scale, void* workspace,
              uint64_t workspace_bytes, cudaStream_t st, double* p95_ttft, double* p95_e2e,
              uint8_t* route, uint16_t* hit, uint64_t* digest, uint64_t* stats, int32_t* cand_status,
              bool host_io, const WindowSpec* win = nullptr, const PolicySpec* pol = nullptr,
              const double* scales = nullptr /* HOST [P] or null */) {
  if (!sim || !params || !workspace || P == 0) return GORGO_ERR_INVALID_ARG;
  if ((!p95_ttft || !p95_e2e) && !win) return GORGO_ERR_INVALID_ARG;
  if (win && (win->window == 0 || win->hop == 0 || win->window > window_max() || !win->best))
    return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  if (win && sim->tr.n_req < win->window) return GORGO_ERR_INVALID_ARG;
  if (!finite_nonneg(scale)) return GORGO_ERR_NONFINITE_PARAM;
  if (scales)
    for (uint32_t p = 0; p < P; ++p)
      if (!finite_nonneg(scales[p])) return GORGO_ERR_NONFINITE_PARAM;
  if ((uintptr_t)workspace % kAlign) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  const Model& m = sim->m;
  const uint64_t N = sim->tr.n_req;
  const bool params_on_device = !host_io && is_device_pointer(params);
  if (!params_on_device && !all_finite(params, (uint64_t)P * m.K)) return GORGO_ERR_NONFINITE_PARAM;

  // largest number of resident candidates the workspace can hold
  uint64_t lo = 0, hi = P;
  while (lo < hi) {
    const uint64_t mid = (lo + hi + 1) / 2;
    if (make_ws(sim, mid, true).total <= workspace_bytes) lo = mid; else hi = mid - 1;
  }
  if (lo == 0) return GORGO_ERR_WORKSPACE_TOO_SMALL;
  const uint32_t res = (uint32_t)lo;
  const WsLayout w = make_ws(sim, res, true);
  unsigned char* base = static_cast<unsigned char*>(workspace);
  double* d_params = reinterpret_cast<double*>(base + w.params);
  double* d_rtt = reinterpret_cast<double*>(base + w.rtt);
  int32_t* d_status = reinterpret_cast<int32_t*>(base + w.status);
  double* d_p95 = reinterpret_cast<double*>(base + w.p95);

  if (cudaMemcpyAsync(d_rtt, sim->rtt.data(), sim->rtt.size() * 8, cudaMemcpyHostToDevice, st) !=
      cudaSuccess)
    return GORGO_ERR_CUDA;
  std::vector<int32_t> h_status;
  if (host_io) h_status.assign(P, 0);
  sim->ev_used = 0;
  sim->wev_used = 0;

  for (uint32_t p0 = 0; p0 < P; p0 += res) {
    const uint32_t pw = (P - p0 < res) ? (P - p0) : res;
    const double* wave_params;
    if (params_on_device) {
      wave_params = params + (size_t)p0 * m.K;
    } else {
      if (cudaMemcpyAsync(d_params, params + (size_t)p0 * m.K, (size_t)pw * m.K * 8,
                          cudaMemcpyHostToDevice, st) != cudaSuccess)
        return GORGO_ERR_CUDA;
      wave_params = d_params;
    }
    if (launch_reset(base + w.masks, (uint64_t)pw * w.mask_stride,
                     reinterpret_cast<uint32_t*>(base + w.exp_head), (uint64_t)pw * N,
                     base + w.states, w.st, m, pw, st) != cudaSuccess)
      return GORGO_ERR_CUDA;
    if (stats && cudaMemsetAsync(stats + (size_t)p0 * 4, 0, (size_t)pw * 32, st) != cudaSuccess)
      return GORGO_ERR_CUDA;

    ReplayArgs a = {};
    a.m = m; a.tr = sim->tr; a.scale = scale;
    if (scales) {
      double* d_scales = reinterpret_cast<double*>(base + w.scales);
      if (cudaMemcpyAsync(d_scales, scales + p0, (size_t)pw * 8, cudaMemcpyHostToDevice, st) !=
          cudaSuccess)
        return GORGO_ERR_CUDA;
      a.scales = d_scales;
    }
    a.first = 0; a.count = (uint32_t)N; a.check_order = 0;
    a.poll_limit = sim->poll_limit; a.ring_polls = sim->ring_polls;
    a.probe_off = sim->probe_off; a.scout_off = sim->scout_off;
    a.rtt = d_rtt; a.params = wave_params;
    a.masks = base + w.masks; a.mask_stride = w.mask_stride;
    a.states = base + w.states; a.lay = w.st;
    a.evict_lists = reinterpret_cast<uint4*>(base + w.lists);
    a.exp_head = reinterpret_cast<uint32_t*>(base + w.exp_head);
    a.exp_rec = reinterpret_cast<uint4*>(base + w.exp_rec);
    a.lru_next = reinterpret_cast<uint32_t*>(base + w.lru_next);
    a.route_log = route ? route + (size_t)p0 * N : base + w.route_log;
    a.route_log_stride = N;
    a.queue_in_requests = pol && pol->queue_in_requests ? 1u : 0u;
    a.forced_route = pol ? pol->forced_route : nullptr;
    if (attach_speeds(sim, base, w, st, &a) != GORGO_OK) return GORGO_ERR_CUDA;
    a.route_out = nullptr;
    a.hit_out = hit ? hit + (size_t)p0 * N : nullptr;
    a.ttft_out = reinterpret_cast<double*>(base + w.ttft);
    a.e2e_out = reinterpret_cast<double*>(base + w.e2e);
    a.out_stride = N;
    a.stats = stats ? stats + (size_t)p0 * 4 : nullptr;
    a.status_out = cand_status ? cand_status + p0 : d_status;
    const bool timed = sim->profiling && sim->ev_used + 2 <= sim->ev.size();
    if (timed && cudaEventRecord(sim->ev[sim->ev_used], st) != cudaSuccess) return GORGO_ERR_CUDA;
    if (launch_replay(a, pw, st) != cudaSuccess) return GORGO_ERR_CUDA;
    if (timed) {
      if (cudaEventRecord(sim->ev[sim->ev_used + 1], st) != cudaSuccess) return GORGO_ERR_CUDA;
      sim->ev_used += 2;
    }

    if (p95_ttft && p95_e2e) {
      SelectArgs s = {};
      s.ttft = a.ttft_out; s.e2e = a.e2e_out; s.stride = N; s.n = (uint32_t)N;
      s.p95_ttft = host_io ? d_p95 : p95_ttft + p0;
      s.p95_e2e = host_io ? d_p95 + res : p95_e2e + p0;
      if (launch_select(s, pw, st) != cudaSuccess) return GORGO_ERR_CUDA;
    }
    if (win) {
      // window values go to the caller's array, else over the E2E scratch (no longer needed)
      WindowArgs wa = {};
      const uint64_t n_win = window_count(N, win->window, win->hop);
      wa.values = a.ttft_out; wa.stride = N;
      wa.window = win->window; wa.hop = win->hop; wa.n_win = (uint32_t)n_win;
      wa.win_p95 = win->win_p95 ? win->win_p95 + (size_t)p0 * n_win : a.e2e_out;
      wa.win_stride = win->win_p95 ? n_win : N;
      wa.best = win->best + p0;
      wa.best_win = win->best_win ? win->best_win + p0 : nullptr;
      const bool wtimed = sim->profiling && sim->wev_used + 2 <= sim->wev.size();
      if (wtimed && cudaEventRecord(sim->wev[sim->wev_used], st) != cudaSuccess) return GORGO_ERR_CUDA;
      if (launch_window(wa, pw, st) != cudaSuccess) return GORGO_ERR_CUDA;
      if (wtimed) {
        if (cudaEventRecord(sim->wev[sim->wev_used + 1], st) != cudaSuccess) return GORGO_ERR_CUDA;
        sim->wev_used += 2;
      }
    }

    if (digest) {
      DigestArgs d = {};
      d.m = m; d.tr = sim->tr; d.states = base + w.states; d.lay = w.st;
      d.route_log = a.route_log; d.route_log_stride = N;
      d.digest = digest + (size_t)p0 * m.R * 2;
      if (launch_digest(d, pw, st) != cudaSuccess) return GORGO_ERR_CUDA;
    }
    if (host_io) {
      if (cudaMemcpyAsync(p95_ttft + p0, d_p95, (size_t)pw * 8, cudaMemcpyDeviceToHost, st) !=
              cudaSuccess ||
          cudaMemcpyAsync(p95_e2e + p0, d_p95 + res, (size_t)pw * 8, cudaMemcpyDeviceToHost, st) !=
              cudaSuccess ||
          cudaMemcpyAsync(h_status.data() + p0, d_status, (size_t)pw * 4, cudaMemcpyDeviceToHost,
                          st) != cudaSuccess)
        return GORGO_ERR_CUDA;
    }
  }
  if (host_io) {
    if (cudaStreamSynchronize(st) != cudaSuccess) return GORGO_ERR_CUDA;
    for (uint32_t p = 0; p < P; ++p)
      if (h_status[p] != 0) return GORGO_ERR_DEVICE_LIMIT;
  }
  return GORGO_OK;
}

}  // namespace

extern "C" {

int gorgo_sim_create(const gorgo_config_t* cfg, gorgo_sim_t** out) {
  if (!cfg || !out || !cfg->rtt_ms) return GORGO_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->n_replicas < 1 || cfg->n_replicas > 64 || cfg->n_regions < 1 ||
      (uint64_t)cfg->n_regions * cfg->n_replicas > 4096 || cfg->slots_per_replica < 1 ||
      cfg->slots_per_replica > 65535 || cfg->block_tokens < 1 || cfg->cache_blocks < 1 ||
      cfg->cache_blocks > 0xFFFFFFF0ull || cfg->reserved != 0)
    return GORGO_ERR_INVALID_ARG;
  if (cfg->n_params != 3 && cfg->n_params != 3 + cfg->n_replicas) return GORGO_ERR_INVALID_ARG;
  if (!finite_nonneg(cfg->prefill_ms_per_token) || !finite_nonneg(cfg->tpot_ms))
    return GORGO_ERR_INVALID_ARG;
  const uint64_t gr = (uint64_t)cfg->n_regions * cfg->n_replicas;
  for (uint64_t i = 0; i < gr; ++i)
    if (!finite_nonneg(cfg->rtt_ms[i])) return GORGO_ERR_INVALID_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess) { cudaGetLastError(); return GORGO_ERR_CUDA; }
  if (cfg->device < 0 || cfg->device >= n_dev) return GORGO_ERR_INVALID_ARG;
  gorgo_sim* s = new (std::nothrow) gorgo_sim();
  if (!s) return GORGO_ERR_INVALID_ARG;
  s->m.R = cfg->n_replicas; s->m.G = cfg->n_regions; s->m.S = cfg->slots_per_replica;
  s->m.B = cfg->block_tokens; s->m.K = cfg->n_params; s->m.C = cfg->cache_blocks;
  s->m.prefill_ms = cfg->prefill_ms_per_token; s->m.tpot_ms = cfg->tpot_ms;
  s->rtt.assign(cfg->rtt_ms, cfg->rtt_ms + gr);
  s->device = cfg->device;
  *out = s;
  return GORGO_OK;
}

int gorgo_sim_destroy(gorgo_sim_t* sim) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  if (!sim->ev.empty()) {
    DeviceGuard guard(sim->device);
    for (cudaEvent_t e : sim->ev) cudaEventDestroy(e);
    for (cudaEvent_t e : sim->wev) cudaEventDestroy(e);
  }
  delete sim;
  return GORGO_OK;
}

int gorgo_sim_set_replica_speeds(gorgo_sim_t* sim, const double* prefill_ms_per_token,
                                 const double* tpot_ms) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  const uint32_t R = sim->m.R;
  for (uint32_t i = 0; i < R; ++i) {
    if (prefill_ms_per_token && !finite_nonneg(prefill_ms_per_token[i])) return GORGO_ERR_INVALID_ARG;
    if (tpot_ms && !finite_nonneg(tpot_ms[i])) return GORGO_ERR_INVALID_ARG;
  }
  if (prefill_ms_per_token) sim->rep_prefill.assign(prefill_ms_per_token, prefill_ms_per_token + R);
  else sim->rep_prefill.clear();
  if (tpot_ms) sim->rep_tpot.assign(tpot_ms, tpot_ms + R);
  else sim->rep_tpot.clear();
  return GORGO_OK;
}

int gorgo_sim_set_proxy_index(gorgo_sim_t* sim, int enable) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  sim->proxy_index = enable ? 1u : 0u;
  return GORGO_OK;
}

int gorgo_sim_set_rtt_series(gorgo_sim_t* sim, uint32_t n_epochs, double epoch_ms, double alpha,
                             const double* samples_ms) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  if (n_epochs == 0) {
    sim->n_epochs = 0; sim->rtt_raw.clear(); sim->rtt_ewma.clear();
    return GORGO_OK;
  }
  if (!samples_ms || !(epoch_ms > 0.0) || !std::isfinite(epoch_ms) || !(alpha > 0.0 && alpha <= 1.0) ||
      n_epochs > (1u << 20))
    return GORGO_ERR_INVALID_ARG;
  const size_t gr = (size_t)sim->m.G * sim->m.R;
  for (size_t x = 0; x < (size_t)n_epochs * gr; ++x)
    if (!finite_nonneg(samples_ms[x])) return GORGO_ERR_INVALID_ARG;
  sim->rtt_raw.assign(samples_ms, samples_ms + (size_t)n_epochs * gr);
  sim->rtt_ewma.assign(samples_ms, samples_ms + (size_t)n_epochs * gr);
  // the proxy's signal: ewma_e = ewma_{e-1} + alpha * (probe_e - ewma_{e-1}), three rounded operations
  for (uint32_t e = 1; e < n_epochs; ++e)
    for (size_t x = 0; x < gr; ++x) {
      const double prev = sim->rtt_ewma[(e - 1) * gr + x];
      const double diff = samples_ms[e * gr + x] - prev;
      const double step = alpha * diff;
      sim->rtt_ewma[e * gr + x] = prev + step;
    }
  sim->n_epochs = n_epochs;
  sim->epoch_ms = epoch_ms;
  return GORGO_OK;
}

int gorgo_sim_set_service_model(gorgo_sim_t* sim, double decode_slowdown, uint64_t kv_budget_tokens) {
  if (!sim || !finite_nonneg(decode_slowdown)) return GORGO_ERR_INVALID_ARG;
  sim->decode_slowdown = decode_slowdown;
  sim->kv_budget = kv_budget_tokens;
  return GORGO_OK;
}

int gorgo_trace_bytes(uint64_t n_requests, uint64_t n_block_ids, uint64_t* bytes_out) {
  if (!bytes_out) return GORGO_ERR_INVALID_ARG;
  *bytes_out = align_up(n_requests * sizeof(ReqRec)) + align_up(n_block_ids * 4) +
               align_up(n_block_ids * 8) + align_up(n_block_ids * 8) + align_up(n_block_ids * 8) +
               align_up(n_requests * 8) +
               align_up((n_requests + 1) * 4) + kAlign;
  return GORGO_OK;
}

// Appends `n_new` requests to the trace under construction in `sim->tb`.  With `atomic` a trace
// that fails a check is left as it was; without it the caller discards the builder on failure.
static int trace_append_impl(gorgo_sim_t* sim, uint64_t n_new, const double* ts_ms,
                             const uint32_t* input_tokens, const uint32_t* output_tokens,
                             const uint16_t* origin, const uint64_t* hash_off,
                             const uint64_t* hash_ids, cudaStream_t st, bool atomic) {
  TraceBuilder& tb = *sim->tb;
  const Model& m = sim->m;
  if (n_new < 1 || hash_off[0] != 0) return GORGO_ERR_BAD_TRACE;
  for (uint64_t k = 0; k < n_new; ++k)
    if (hash_off[k + 1] < hash_off[k]) return GORGO_ERR_BAD_TRACE;
  const uint64_t Tn = hash_off[n_new];
  const uint64_t N0 = tb.N, T0 = tb.T, N = N0 + n_new, T = T0 + Tn;
  if (N > tb.cap_req || T > tb.cap_ids) return GORGO_ERR_WORKSPACE_TOO_SMALL;
  if (Tn > 0 && !hash_ids) return GORGO_ERR_INVALID_ARG;
  const uint64_t nmax = m.C < 65535 ? m.C : 65535;

  std::vector<ReqRec> req(n_new);
  double prev_t = N0 ? tb.ts.back() : 0.0;
  for (uint64_t k = 0; k < n_new; ++k) {
    const double t = ts_ms[k];
    if (!finite_nonneg(t) || t < prev_t) return GORGO_ERR_BAD_TRACE;
    prev_t = t;
    const uint64_t n = hash_off[k + 1] - hash_off[k];
    const uint64_t want = ((uint64_t)input_tokens[k] + m.B - 1) / m.B;
    if (n != want || n > nmax) return GORGO_ERR_BAD_TRACE;
    const uint16_t g = origin ? origin[k] : (uint16_t)0;
    if (g >= m.G) return GORGO_ERR_BAD_TRACE;
    ReqRec& q = req[k];
    q.ts_ms = t; q.off = (uint32_t)(T0 + hash_off[k]); q.in_tok = input_tokens[k];
    q.out_tok = output_tokens[k]; q.nblk = (uint16_t)n; q.origin = g; q.prev_share = kNone; q.pad = 0;
  }
  if (atomic) {   // an id twice in one request: found before anything is changed
    std::vector<uint64_t> tmp;
    for (uint64_t k = 0; k < n_new; ++k) {
      tmp.assign(hash_ids + hash_off[k], hash_ids + hash_off[k + 1]);
      std::sort(tmp.begin(), tmp.end());
      if (std::adjacent_find(tmp.begin(), tmp.end()) != tmp.end()) return GORGO_ERR_BAD_TRACE;
    }
  }

  // dense renumbering in order of first appearance; per block the previous occurrence, and the
  // next one where that lies in this batch (an earlier batch's entry is patched on the device)
  std::vector<uint32_t> ids(Tn);
  std::vector<uint2> occ(Tn, make_uint2(kNone, kNone)), occ_before(Tn);
  const uint32_t D0 = tb.D;
  bool patch_old = false;
  for (uint64_t k = 0; k < n_new; ++k) {
    const uint32_t r = (uint32_t)(N0 + k);
    uint32_t latest = 0;  // latest earlier request (+1) that contains one of this one's blocks
    for (uint64_t gl = hash_off[k]; gl < hash_off[k + 1]; ++gl) {
      const uint32_t before = tb.D;
      const uint32_t d = tb.map.get_or_add(hash_ids[gl], tb.D);
      if (tb.D != before) {
        tb.raw_new.push_back(hash_ids[gl]);
        tb.seen_in.push_back(0); tb.last_g.push_back(kNone); tb.last_r.push_back(kNone);
      }
      if (tb.seen_in[d] == r + 1) return GORGO_ERR_BAD_TRACE;   // (not reached when `atomic`)
      if (tb.seen_in[d] > latest) latest = tb.seen_in[d];
      tb.seen_in[d] = r + 1;
      ids[gl] = d;
      const uint32_t g = (uint32_t)(T0 + gl);
      const uint32_t pg = tb.last_g[d];
      occ_before[gl] = make_uint2(pg, tb.last_r[d]);
      if (pg != kNone) {
        if (pg >= T0) occ[pg - T0] = make_uint2(g, r);
        else patch_old = true;
      }
      tb.last_g[d] = g; tb.last_r[d] = r;
    }
    req[k].prev_share = latest ? latest - 1 : kNone;
  }
  tb.ts.insert(tb.ts.end(), ts_ms, ts_ms + n_new);

  // time grid over the arrivals: grid[b] = first request with ts >= b * dt (the last request if
  // there is none), b = 0..n_grid; none while all requests arrive at one instant.  The first
  // build takes about one request per bucket; later batches add buckets of the same width.
  // Entries written earlier stay valid: the replay only needs a lower bound of the request it
  // searches for.
  std::vector<uint32_t> grid;
  uint32_t grid_from = 0;
  {
    const double span = tb.ts.back();
    const double buckets = tb.grid_n ? std::floor(span / tb.grid_dt) : 0.0;
    if (tb.grid_n == 0 || buckets > (double)tb.cap_req) {
      const double dt = span / (double)N;
      tb.grid_n = 0; tb.grid_dt = 0.0;
      if (dt > 0.0 && std::isfinite(dt) && dt >= span * 0x1p-40) {
        tb.grid_n = (uint32_t)N; tb.grid_dt = dt;
        grid.resize((size_t)N + 1);
        uint64_t r = 0;
        for (uint32_t b = 0; b <= tb.grid_n; ++b) {
          const double edge = (double)b * dt;
          while (r < N && tb.ts[r] < edge) ++r;
          grid[b] = (uint32_t)(r < N ? r : N - 1);
        }
        tb.grid_cursor = r;
      }
    } else if ((uint32_t)buckets > tb.grid_n) {
      grid_from = tb.grid_n + 1;
      const uint32_t upto = (uint32_t)buckets;
      grid.resize(upto - tb.grid_n);
      uint64_t r = tb.grid_cursor;
      for (uint32_t b = grid_from; b <= upto; ++b) {
        const double edge = (double)b * tb.grid_dt;
        while (r < N && tb.ts[r] < edge) ++r;
        grid[b - grid_from] = (uint32_t)(r < N ? r : N - 1);
      }
      tb.grid_cursor = r;
      tb.grid_n = upto;
    }
  }

  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  const uint64_t Dn = tb.D - D0;
  bool ok = cudaMemcpyAsync(tb.d_req + N0 * sizeof(ReqRec), req.data(), n_new * sizeof(ReqRec),
                            cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(tb.d_ts + N0 * 8, ts_ms, n_new * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!grid.empty())
    ok = ok && cudaMemcpyAsync(tb.d_grid + (size_t)grid_from * 4, grid.data(), grid.size() * 4,
                               cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (Tn > 0) {
    ok = ok && cudaMemcpyAsync(tb.d_ids + T0 * 4, ids.data(), Tn * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(tb.d_occ + T0 * 8, occ.data(), Tn * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(tb.d_prev + T0 * 8, occ_before.data(), Tn * 8, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (Dn > 0)
      ok = ok && cudaMemcpyAsync(tb.d_raw + (size_t)D0 * 8, tb.raw_new.data(), Dn * 8,
                                 cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  tb.raw_new.clear();
  tb.N = N; tb.T = T;
  if (!ok) { cudaGetLastError(); sim->has_trace = false; return GORGO_ERR_CUDA; }
  sim->tr.req = reinterpret_cast<const ReqRec*>(tb.d_req);
  sim->tr.ids = reinterpret_cast<const uint32_t*>(tb.d_ids);
  sim->tr.occ_next = reinterpret_cast<const uint2*>(tb.d_occ);
  sim->tr.occ_prev = reinterpret_cast<const uint2*>(tb.d_prev);
  sim->tr.raw_id = reinterpret_cast<const uint64_t*>(tb.d_raw);
  sim->tr.ts = reinterpret_cast<const double*>(tb.d_ts);
  sim->tr.grid = reinterpret_cast<const uint32_t*>(tb.d_grid);
  sim->tr.grid_dt = tb.grid_dt;
  sim->tr.grid_n = tb.grid_n;
  sim->tr.n_req = (uint32_t)N; sim->tr.n_ids = (uint32_t)T; sim->tr.n_distinct = tb.D;
  // earlier batches' last occurrences now have a successor
  if (patch_old && launch_link_occurrences(sim->tr, (uint32_t)N0, (uint32_t)n_new, (uint32_t)T0,
                                           reinterpret_cast<uint2*>(tb.d_occ), st) != cudaSuccess) {
    sim->has_trace = false;
    return GORGO_ERR_CUDA;
  }
  sim->has_trace = true;
  return GORGO_OK;
}

static int trace_begin_impl(gorgo_sim_t* sim, uint64_t max_requests, uint64_t max_block_ids,
                            void* dev_trace_buf, uint64_t dev_trace_bytes) {
  if (!sim || !dev_trace_buf) return GORGO_ERR_INVALID_ARG;
  if ((uintptr_t)dev_trace_buf % kAlign) return GORGO_ERR_INVALID_ARG;
  if (max_requests < 1 || max_requests >= 0xFFFFFFFFull || max_block_ids >= 0xFFFFFFFFull)
    return GORGO_ERR_BAD_TRACE;
  uint64_t need = 0;
  gorgo_trace_bytes(max_requests, max_block_ids, &need);
  if (dev_trace_bytes < need) return GORGO_ERR_WORKSPACE_TOO_SMALL;
  sim->has_trace = false;
  sim->tr = TraceView{};
  sim->cap_req = sim->cap_ids = 0;
  sim->tb.reset(new TraceBuilder());
  TraceBuilder& tb = *sim->tb;
  tb.cap_req = max_requests; tb.cap_ids = max_block_ids;
  const uint64_t N = max_requests, T = max_block_ids;
  unsigned char* base = static_cast<unsigned char*>(dev_trace_buf);
  uint64_t o = 0;
  tb.d_req = base + o; o += align_up(N * sizeof(ReqRec));
  tb.d_ids = base + o; o += align_up(T * 4);
  tb.d_occ = base + o; o += align_up(T * 8);
  tb.d_raw = base + o; o += align_up(T * 8);
  tb.d_prev = base + o; o += align_up(T * 8);
  tb.d_ts = base + o; o += align_up(N * 8);
  tb.d_grid = base + o; o += align_up((N + 1) * 4);
  return GORGO_OK;
}

int gorgo_trace_upload(gorgo_sim_t* sim, uint64_t n_requests, const double* ts_ms,
                       const uint32_t* input_tokens, const uint32_t* output_tokens,
                       const uint16_t* origin, const uint64_t* hash_off, const uint64_t* hash_ids,
                       void* dev_trace_buf, uint64_t dev_trace_bytes, void* cuda_stream) {
  if (!sim || !ts_ms || !input_tokens || !output_tokens || !hash_off || !dev_trace_buf)
    return GORGO_ERR_INVALID_ARG;
  if (n_requests < 1 || n_requests >= 0xFFFFFFFFull) return GORGO_ERR_BAD_TRACE;
  if (hash_off[0] != 0) return GORGO_ERR_BAD_TRACE;
  for (uint64_t r = 0; r < n_requests; ++r)
    if (hash_off[r + 1] < hash_off[r]) return GORGO_ERR_BAD_TRACE;
  // a fixed trace is an appendable one of exactly its own size, built in one batch
  int rc = trace_begin_impl(sim, n_requests, hash_off[n_requests], dev_trace_buf, dev_trace_bytes);
  if (rc == GORGO_OK) {
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    rc = trace_append_impl(sim, n_requests, ts_ms, input_tokens, output_tokens, origin, hash_off,
                           hash_ids, st, false);
    if (rc == GORGO_OK) {
      DeviceGuard guard(sim->device);
      if (!guard.ok || cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); rc = GORGO_ERR_CUDA; }
    }
  }
  sim->tb.reset();           // nothing can be appended to an uploaded trace
  if (rc != GORGO_OK) sim->has_trace = false;
  return rc;
}

int gorgo_trace_begin(gorgo_sim_t* sim, uint64_t max_requests, uint64_t max_block_ids,
                      void* dev_trace_buf, uint64_t dev_trace_bytes) {
  const int rc = trace_begin_impl(sim, max_requests, max_block_ids, dev_trace_buf, dev_trace_bytes);
  if (rc == GORGO_OK) { sim->cap_req = max_requests; sim->cap_ids = max_block_ids; }
  return rc;
}

int gorgo_trace_append(gorgo_sim_t* sim, uint64_t n_requests, const double* ts_ms,
                       const uint32_t* input_tokens, const uint32_t* output_tokens,
                       const uint16_t* origin, const uint64_t* hash_off, const uint64_t* hash_ids,
                       void* cuda_stream) {
  if (!sim || !ts_ms || !input_tokens || !output_tokens || !hash_off) return GORGO_ERR_INVALID_ARG;
  if (!sim->tb) return GORGO_ERR_NO_TRACE;
  return trace_append_impl(sim, n_requests, ts_ms, input_tokens, output_tokens, origin, hash_off,
                           hash_ids, static_cast<cudaStream_t>(cuda_stream), true);
}

int gorgo_trace_info(const gorgo_sim_t* sim, uint64_t* n_requests, uint64_t* n_block_ids,
                     uint64_t* n_distinct) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  if (n_requests) *n_requests = sim->tr.n_req;
  if (n_block_ids) *n_block_ids = sim->tr.n_ids;
  if (n_distinct) *n_distinct = sim->tr.n_distinct;
  return GORGO_OK;
}

int gorgo_workspace_bytes(const gorgo_sim_t* sim, uint32_t resident_candidates,
                          uint64_t* bytes_out) {
  if (!sim || !bytes_out || resident_candidates == 0) return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  *bytes_out = make_ws(sim, resident_candidates, true).total;
  return GORGO_OK;
}

int gorgo_eval_population(gorgo_sim_t* sim, uint32_t n_candidates, const double* params,
                          double time_scale, void* workspace, uint64_t workspace_bytes,
                          void* cuda_stream, double* p95_ttft_ms, double* p95_e2e_ms,
                          uint8_t* route, uint16_t* hit_blocks, uint64_t* state_digest,
                          uint64_t* stats, int32_t* cand_status) {
  return eval_impl(sim, n_candidates, params, time_scale, workspace, workspace_bytes,
                   static_cast<cudaStream_t>(cuda_stream), p95_ttft_ms, p95_e2e_ms, route,
                   hit_blocks, state_digest, stats, cand_status, false);
}

int gorgo_eval_population_scales(gorgo_sim_t* sim, uint32_t n_candidates, const double* params,
                                 const double* time_scales, void* workspace,
                                 uint64_t workspace_bytes, void* cuda_stream, double* p95_ttft_ms,
                                 double* p95_e2e_ms, uint8_t* route, uint16_t* hit_blocks,
                                 uint64_t* state_digest, int32_t* cand_status) {
  if (!time_scales) return GORGO_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int rc = eval_impl(sim, n_candidates, params, 1.0, workspace, workspace_bytes, st,
                           p95_ttft_ms, p95_e2e_ms, route, hit_blocks, state_digest, nullptr,
                           cand_status, false, nullptr, nullptr, time_scales);
  // `time_scales` is host memory read by asynchronous copies
  if (rc == GORGO_OK && cudaStreamSynchronize(st) != cudaSuccess) return GORGO_ERR_CUDA;
  return rc;
}

int gorgo_eval_population_windows(gorgo_sim_t* sim, uint32_t n_candidates, const double* params,
                                  double time_scale, void* workspace, uint64_t workspace_bytes,
                                  void* cuda_stream, uint32_t window, uint32_t hop,
                                  double* win_p95_ttft_ms, double* best_win_p95_ttft_ms,
                                  uint32_t* best_window, double* p95_ttft_ms, double* p95_e2e_ms,
                                  int32_t* cand_status) {
  WindowSpec w = {window, hop, win_p95_ttft_ms, best_win_p95_ttft_ms, best_window};
  if ((p95_ttft_ms == nullptr) != (p95_e2e_ms == nullptr)) return GORGO_ERR_INVALID_ARG;
  return eval_impl(sim, n_candidates, params, time_scale, workspace, workspace_bytes,
                   static_cast<cudaStream_t>(cuda_stream), p95_ttft_ms, p95_e2e_ms, nullptr, nullptr,
                   nullptr, nullptr, cand_status, false, &w);
}

int gorgo_eval_policy(gorgo_sim_t* sim, uint32_t policy, const uint32_t* draws, double time_scale,
                      void* workspace, uint64_t workspace_bytes, void* cuda_stream,
                      double* p95_ttft_ms, double* p95_e2e_ms, uint8_t* route, uint16_t* hit_blocks,
                      uint64_t* state_digest, int32_t* cand_status) {
  if (!sim || !workspace || policy > GORGO_POLICY_RANDOM) return GORGO_ERR_INVALID_ARG;
  if (policy == GORGO_POLICY_RANDOM && !draws) return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  if ((uintptr_t)workspace % kAlign) return GORGO_ERR_INVALID_ARG;
  const WsLayout w = make_ws(sim, 1, true);
  if (w.total > workspace_bytes) return GORGO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* base = static_cast<unsigned char*>(workspace);
  const uint32_t K = sim->m.K;
  // weights of the named policy: (w_net, w_prefill, w_queue), normalisers 1
  std::vector<double> wts(K, 0.0);
  for (uint32_t k = 3; k < K; ++k) wts[k] = 1.0;
  PolicySpec ps = {false, nullptr};
  switch (policy) {
    case GORGO_POLICY_LEAST_LOAD: wts[2] = 1.0; break;
    case GORGO_POLICY_LEAST_REQUEST: wts[2] = 1.0; ps.queue_in_requests = true; break;
    case GORGO_POLICY_PREFIX_CACHE: wts[1] = 1.0; break;
    default: {
      DeviceGuard guard(sim->device);
      if (!guard.ok) return GORGO_ERR_CUDA;
      uint8_t* d_forced = base + w.forced;
      uint32_t* d_draws = reinterpret_cast<uint32_t*>(base + w.draws);
      const bool affinity = policy == GORGO_POLICY_SESSION_AFFINITY;
      if (!affinity && cudaMemcpyAsync(d_draws, draws, (size_t)sim->tr.n_req * 4,
                                       cudaMemcpyHostToDevice, st) != cudaSuccess)
        return GORGO_ERR_CUDA;
      if (launch_policy_routes(sim->tr, sim->m.R, affinity, d_draws, d_forced, st) != cudaSuccess)
        return GORGO_ERR_CUDA;
      ps.forced_route = d_forced;
    }
  }
  const int rc = eval_impl(sim, 1, wts.data(), time_scale, workspace, workspace_bytes, st,
                           p95_ttft_ms, p95_e2e_ms, route, hit_blocks, state_digest, nullptr,
                           cand_status, false, nullptr, &ps);
  // `wts` and the caller's `draws` are host memory read by asynchronous copies
  if (rc == GORGO_OK && cudaStreamSynchronize(st) != cudaSuccess) return GORGO_ERR_CUDA;
  return rc;
}

int gorgo_window_count(uint64_t n_requests, uint32_t window, uint32_t hop, uint64_t* n_windows) {
  if (!n_windows || window == 0 || hop == 0) return GORGO_ERR_INVALID_ARG;
  *n_windows = window_count(n_requests, window, hop);
  return GORGO_OK;
}

int gorgo_eval_population_host(gorgo_sim_t* sim, uint32_t n_candidates, const double* params,
                               double time_scale, void* workspace, uint64_t workspace_bytes,
                               void* cuda_stream, double* p95_ttft_ms, double* p95_e2e_ms) {
  return eval_impl(sim, n_candidates, params, time_scale, workspace, workspace_bytes,
                   static_cast<cudaStream_t>(cuda_stream), p95_ttft_ms, p95_e2e_ms, nullptr,
                   nullptr, nullptr, nullptr, nullptr, true);
}

// (1+lambda) evolution strategy of the paper's tuner (Section 2.3, Eq. 4) on top of the batched
// evaluator: every step mutates the parent lambda times, replays all offspring in one population
// evaluation, and keeps the best one if it beats the parent.  Host logic only; the replays and
// their p95 reduction run on the device.
int gorgo_es_run(gorgo_sim_t* sim, const gorgo_es_config_t* cfg, const double* x0, const double* z,
                 void* workspace, uint64_t workspace_bytes, void* cuda_stream, double* x_best,
                 double* objective_best, double* sigma_final, double* history) {
  if (!sim || !cfg || !x0 || !z || !workspace || !x_best || !objective_best || !sigma_final)
    return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  const uint32_t K = sim->m.K, T = cfg->n_tuned, L = cfg->lambda;
  if (L == 0 || T == 0 || T > K || !cfg->tuned || !cfg->lo || !cfg->hi || cfg->objective > 1)
    return GORGO_ERR_INVALID_ARG;
  if (!(cfg->sigma0 > 0.0) || !std::isfinite(cfg->sigma0) || !(cfg->sigma_up > 1.0) ||
      !std::isfinite(cfg->sigma_up))
    return GORGO_ERR_NONFINITE_PARAM;
  if (!all_finite(x0, K) || !all_finite(z, (uint64_t)cfg->n_steps * L * T))
    return GORGO_ERR_NONFINITE_PARAM;
  for (uint32_t k = 0; k < T; ++k) {
    if (cfg->tuned[k] >= K) return GORGO_ERR_INVALID_ARG;
    if (!(cfg->lo[k] > 0.0) || !(cfg->hi[k] >= cfg->lo[k]) || !std::isfinite(cfg->hi[k]))
      return GORGO_ERR_INVALID_ARG;
    if (!(x0[cfg->tuned[k]] > 0.0)) return GORGO_ERR_INVALID_ARG;   // ln(x) of Eq. 4
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  std::vector<double> parent(x0, x0 + K), pop((size_t)L * K), pt(L), pe(L);
  // the parent's own objective
  double ft = 0.0, fe = 0.0;
  int rc = eval_impl(sim, 1, parent.data(), cfg->time_scale, workspace, workspace_bytes, st, &ft,
                     &fe, nullptr, nullptr, nullptr, nullptr, nullptr, true);
  if (rc != GORGO_OK) return rc;
  double f_parent = cfg->objective == 0 ? ft : fe;
  double sigma = cfg->sigma0;
  const double down = std::pow(cfg->sigma_up, -0.25);   // one success in five keeps sigma in place
  for (uint32_t t = 0; t < cfg->n_steps; ++t) {
    for (uint32_t l = 0; l < L; ++l) {
      double* x = pop.data() + (size_t)l * K;
      std::copy(parent.begin(), parent.end(), x);
      for (uint32_t k = 0; k < T; ++k) {
        const double step = sigma * z[((size_t)t * L + l) * T + k];
        double v = std::exp(std::log(parent[cfg->tuned[k]]) + step);     // Eq. 4
        if (v < cfg->lo[k]) v = cfg->lo[k];
        if (v > cfg->hi[k]) v = cfg->hi[k];
        x[cfg->tuned[k]] = v;
      }
    }
    rc = eval_impl(sim, L, pop.data(), cfg->time_scale, workspace, workspace_bytes, st, pt.data(),
                   pe.data(), nullptr, nullptr, nullptr, nullptr, nullptr, true);
    if (rc != GORGO_OK) return rc;
    const std::vector<double>& f = cfg->objective == 0 ? pt : pe;
    uint32_t best = 0;
    for (uint32_t l = 1; l < L; ++l)
      if (f[l] < f[best]) best = l;                 // lowest index among equals
    const bool accept = f[best] < f_parent;         // the offspring has to beat the parent
    const double f_best = f[best];
    if (accept) {
      std::copy(pop.begin() + (size_t)best * K, pop.begin() + (size_t)(best + 1) * K, parent.begin());
      f_parent = f_best;
      sigma *= cfg->sigma_up;
    } else {
      sigma *= down;
    }
    if (history) {
      double* h = history + (size_t)t * (4 + T);
      h[0] = f_best; h[1] = accept ? 1.0 : 0.0; h[2] = sigma; h[3] = f_parent;
      for (uint32_t k = 0; k < T; ++k) h[4 + k] = parent[cfg->tuned[k]];
    }
  }
  std::copy(parent.begin(), parent.end(), x_best);
  *objective_best = f_parent;
  *sigma_final = sigma;
  return GORGO_OK;
}

// Online (1+1)-ES inside one replay (paper Section 2.3 and Section 4): P independent tuners, each on
// its own simulator state, all advanced together: one replay launch per chunk of requests (the
// first `window`, then `hop` at a time), one launch that reduces the last `window` TTFTs of
// every tuner to their p95, and the strategy's step on the host (Eq. 4 with the C library's exp
// and log, like gorgo_es_run).  No step of the simulation runs on the host.
int gorgo_tune_online(gorgo_sim_t* sim, const gorgo_online_config_t* cfg, uint32_t n_tuners,
                      const double* x0, const double* z, void* workspace, uint64_t workspace_bytes,
                      void* cuda_stream, double* x_final, double* sigma_final, uint32_t* steps_done,
                      double* history, double* p95_ttft_ms, double* p95_e2e_ms, uint8_t* route) {
  if (!sim || !cfg || !x0 || !workspace || !x_final || !sigma_final || n_tuners == 0)
    return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  const uint32_t K = sim->m.K, T = cfg->n_tuned, P = n_tuners;
  const uint64_t N = sim->tr.n_req;
  if (T == 0 || T > K || !cfg->tuned || !cfg->lo || !cfg->hi || cfg->window == 0 || cfg->hop == 0 ||
      cfg->window > window_max() || (cfg->n_draw_steps > 0 && !z))
    return GORGO_ERR_INVALID_ARG;
  if (!(cfg->sigma0 > 0.0) || !std::isfinite(cfg->sigma0) || !(cfg->sigma_up > 1.0) ||
      !std::isfinite(cfg->sigma_up) || !finite_nonneg(cfg->time_scale))
    return GORGO_ERR_NONFINITE_PARAM;
  if (!all_finite(x0, (uint64_t)P * K) || !all_finite(z, (uint64_t)P * cfg->n_draw_steps * T))
    return GORGO_ERR_NONFINITE_PARAM;
  for (uint32_t k = 0; k < T; ++k) {
    if (cfg->tuned[k] >= K) return GORGO_ERR_INVALID_ARG;
    if (!(cfg->lo[k] > 0.0) || !(cfg->hi[k] >= cfg->lo[k]) || !std::isfinite(cfg->hi[k]))
      return GORGO_ERR_INVALID_ARG;
    for (uint32_t p = 0; p < P; ++p)
      if (!(x0[(size_t)p * K + cfg->tuned[k]] > 0.0)) return GORGO_ERR_INVALID_ARG;   // ln(x) of Eq. 4
  }
  if ((uintptr_t)workspace % kAlign) return GORGO_ERR_INVALID_ARG;
  const WsLayout w = make_ws(sim, P, true);                 // every tuner's state stays resident
  if (w.total > workspace_bytes) return GORGO_ERR_WORKSPACE_TOO_SMALL;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* base = static_cast<unsigned char*>(workspace);
  double* d_params = reinterpret_cast<double*>(base + w.params);
  double* d_rtt = reinterpret_cast<double*>(base + w.rtt);
  int32_t* d_status = reinterpret_cast<int32_t*>(base + w.status);
  double* d_p95 = reinterpret_cast<double*>(base + w.p95);
  double* d_ttft = reinterpret_cast<double*>(base + w.ttft);
  double* d_e2e = reinterpret_cast<double*>(base + w.e2e);
  if (cudaMemcpyAsync(d_rtt, sim->rtt.data(), sim->rtt.size() * 8, cudaMemcpyHostToDevice, st) !=
          cudaSuccess ||
      cudaMemsetAsync(d_status, 0, (size_t)P * 4, st) != cudaSuccess)
    return GORGO_ERR_CUDA;
  if (launch_reset(base + w.masks, (uint64_t)P * w.mask_stride,
                   reinterpret_cast<uint32_t*>(base + w.exp_head), (uint64_t)P * N, base + w.states,
                   w.st, sim->m, P, st) != cudaSuccess)
    return GORGO_ERR_CUDA;

  std::vector<double> parent(x0, x0 + (size_t)P * K), live(parent), f_parent(P, 0.0), sigma(P, cfg->sigma0),
      value(P, 0.0);
  const double down = std::pow(cfg->sigma_up, -0.25);   // one success in five keeps sigma in place
  const uint32_t hist_w = 4 + 2 * T;
  uint64_t done = 0;
  uint32_t step = 0;
  while (done < N) {
    const uint64_t count = std::min<uint64_t>(done == 0 ? cfg->window : cfg->hop, N - done);
    if (cudaMemcpyAsync(d_params, live.data(), (size_t)P * K * 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return GORGO_ERR_CUDA;
    ReplayArgs a = {};
    a.m = sim->m; a.tr = sim->tr; a.scale = cfg->time_scale;
    a.first = (uint32_t)done; a.count = (uint32_t)count; a.check_order = 1;
    a.poll_limit = sim->poll_limit; a.ring_polls = sim->ring_polls;
    a.probe_off = sim->probe_off; a.scout_off = sim->scout_off;
    a.rtt = d_rtt; a.params = d_params;
    a.masks = base + w.masks; a.mask_stride = w.mask_stride;
    a.states = base + w.states; a.lay = w.st;
    a.evict_lists = reinterpret_cast<uint4*>(base + w.lists);
    a.exp_head = reinterpret_cast<uint32_t*>(base + w.exp_head);
    a.exp_rec = reinterpret_cast<uint4*>(base + w.exp_rec);
    a.lru_next = reinterpret_cast<uint32_t*>(base + w.lru_next);
    a.route_log = route ? route : base + w.route_log;
    a.route_log_stride = N;
    if (attach_speeds(sim, base, w, st, &a) != GORGO_OK) return GORGO_ERR_CUDA;
    a.ttft_out = d_ttft + done; a.e2e_out = d_e2e + done; a.out_stride = N;   // request r at [p*N + r]
    a.status_out = d_status;
    if (launch_replay(a, P, st) != cudaSuccess) return GORGO_ERR_CUDA;
    done += count;
    // a strategy step where a full window ends and draws are left
    if (done < cfg->window || (done - cfg->window) % cfg->hop != 0 || step >= cfg->n_draw_steps)
      continue;                                   // (`live` is unchanged: nothing to wait for)
    WindowArgs wa = {};
    wa.values = d_ttft + (done - cfg->window); wa.stride = N;
    wa.window = cfg->window; wa.hop = cfg->hop; wa.n_win = 1;
    wa.win_p95 = d_p95; wa.win_stride = 1;
    wa.best = d_p95 + P; wa.best_win = nullptr;
    if (launch_window(wa, P, st) != cudaSuccess) return GORGO_ERR_CUDA;
    if (cudaMemcpyAsync(value.data(), d_p95 + P, (size_t)P * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
      return GORGO_ERR_CUDA;
    for (uint32_t p = 0; p < P; ++p) {
      double* par = parent.data() + (size_t)p * K;
      double* lv = live.data() + (size_t)p * K;
      bool accept = false;
      if (step == 0) {
        f_parent[p] = value[p];                             // the start weights themselves
      } else {
        accept = value[p] < f_parent[p];
        if (accept) {
          std::copy(lv, lv + K, par);
          f_parent[p] = value[p];
          sigma[p] *= cfg->sigma_up;
        } else {
          sigma[p] *= down;
        }
      }
      std::copy(par, par + K, lv);
      for (uint32_t k = 0; k < T; ++k) {
        const double zk = z[((size_t)p * cfg->n_draw_steps + step) * T + k];
        const double stepv = sigma[p] * zk;
        double v = std::exp(std::log(par[cfg->tuned[k]]) + stepv);     // Eq. 4
        if (v < cfg->lo[k]) v = cfg->lo[k];
        if (v > cfg->hi[k]) v = cfg->hi[k];
        lv[cfg->tuned[k]] = v;
      }
      if (history) {
        double* h = history + ((size_t)p * cfg->n_draw_steps + step) * hist_w;
        h[0] = value[p]; h[1] = accept ? 1.0 : 0.0; h[2] = sigma[p]; h[3] = f_parent[p];
        for (uint32_t k = 0; k < T; ++k) { h[4 + k] = par[cfg->tuned[k]]; h[4 + T + k] = lv[cfg->tuned[k]]; }
      }
    }
    ++step;
  }
  if (p95_ttft_ms && p95_e2e_ms) {
    SelectArgs sa = {};
    sa.ttft = d_ttft; sa.e2e = d_e2e; sa.stride = N; sa.n = (uint32_t)N;
    sa.p95_ttft = d_p95; sa.p95_e2e = d_p95 + P;
    if (launch_select(sa, P, st) != cudaSuccess) return GORGO_ERR_CUDA;
    if (cudaMemcpyAsync(p95_ttft_ms, d_p95, (size_t)P * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(p95_e2e_ms, d_p95 + P, (size_t)P * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess)
      return GORGO_ERR_CUDA;
  }
  std::vector<int32_t> h_status(P, 0);
  if (cudaMemcpyAsync(h_status.data(), d_status, (size_t)P * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return GORGO_ERR_CUDA;
  std::copy(parent.begin(), parent.end(), x_final);
  std::copy(sigma.begin(), sigma.end(), sigma_final);
  if (steps_done) *steps_done = step;
  for (uint32_t p = 0; p < P; ++p)
    if (h_status[p] != 0) return h_status[p] == -8 ? GORGO_ERR_OUT_OF_ORDER : GORGO_ERR_DEVICE_LIMIT;
  return GORGO_OK;
}

int gorgo_state_bytes(const gorgo_sim_t* sim, uint64_t* bytes_out) {
  if (!sim || !bytes_out) return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  *bytes_out = make_ws(sim, 1, false).total;
  return GORGO_OK;
}

static int state_check(gorgo_sim_t* sim, void* ws, uint64_t bytes, WsLayout* w) {
  if (!sim || !ws) return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  if ((uintptr_t)ws % kAlign) return GORGO_ERR_INVALID_ARG;
  *w = make_ws(sim, 1, false);
  if (bytes < w->total) return GORGO_ERR_WORKSPACE_TOO_SMALL;
  return GORGO_OK;
}

int gorgo_sim_reset(gorgo_sim_t* sim, void* state_workspace, uint64_t state_bytes,
                    void* cuda_stream) {
  WsLayout w;
  const int rc = state_check(sim, state_workspace, state_bytes, &w);
  if (rc != GORGO_OK) return rc;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  unsigned char* base = static_cast<unsigned char*>(state_workspace);
  if (launch_reset(base + w.masks, w.mask_stride, reinterpret_cast<uint32_t*>(base + w.exp_head),
                   sim->cap_req ? sim->cap_req : sim->tr.n_req, base + w.states, w.st, sim->m, 1,
                   static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return GORGO_ERR_CUDA;
  return GORGO_OK;
}

int gorgo_route_batch(gorgo_sim_t* sim, const double* params, double time_scale, uint64_t first,
                      uint64_t count, void* state_workspace, uint64_t state_bytes,
                      void* cuda_stream, uint8_t* route, uint16_t* hit_blocks, double* ttft_ms,
                      double* e2e_ms) {
  WsLayout w;
  const int rc = state_check(sim, state_workspace, state_bytes, &w);
  if (rc != GORGO_OK) return rc;
  if (!params || !route) return GORGO_ERR_INVALID_ARG;
  const uint64_t N = sim->tr.n_req;
  if (first > N || count > N - first) return GORGO_ERR_INVALID_ARG;
  if (!finite_nonneg(time_scale) || !all_finite(params, sim->m.K)) return GORGO_ERR_NONFINITE_PARAM;
  if (count == 0) return GORGO_OK;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* base = static_cast<unsigned char*>(state_workspace);
  double* d_params = reinterpret_cast<double*>(base + w.params);
  double* d_rtt = reinterpret_cast<double*>(base + w.rtt);
  if (cudaMemcpyAsync(d_rtt, sim->rtt.data(), sim->rtt.size() * 8, cudaMemcpyHostToDevice, st) !=
          cudaSuccess ||
      cudaMemcpyAsync(d_params, params, (size_t)sim->m.K * 8, cudaMemcpyHostToDevice, st) !=
          cudaSuccess)
    return GORGO_ERR_CUDA;
  ReplayArgs a = {};
  a.m = sim->m; a.tr = sim->tr; a.scale = time_scale;
  a.first = (uint32_t)first; a.count = (uint32_t)count; a.check_order = 1;
  a.poll_limit = sim->poll_limit; a.ring_polls = sim->ring_polls;
  a.probe_off = sim->probe_off; a.scout_off = sim->scout_off;
  a.rtt = d_rtt; a.params = d_params;
  a.masks = base + w.masks; a.mask_stride = w.mask_stride;
  a.states = base + w.states; a.lay = w.st;
  a.evict_lists = reinterpret_cast<uint4*>(base + w.lists);
  a.exp_head = reinterpret_cast<uint32_t*>(base + w.exp_head);
  a.exp_rec = reinterpret_cast<uint4*>(base + w.exp_rec);
  a.lru_next = reinterpret_cast<uint32_t*>(base + w.lru_next);
  a.route_log = base + w.route_log; a.route_log_stride = N;
  a.finish_log = reinterpret_cast<double*>(base + w.finish);
  if (attach_speeds(sim, base, w, st, &a) != GORGO_OK) return GORGO_ERR_CUDA;
  a.route_out = route; a.hit_out = hit_blocks; a.ttft_out = ttft_ms; a.e2e_out = e2e_ms;
  a.out_stride = count;
  a.stats = nullptr; a.status_out = nullptr;
  if (launch_replay(a, 1, st) != cudaSuccess) return GORGO_ERR_CUDA;
  return GORGO_OK;
}

int gorgo_state_digest(gorgo_sim_t* sim, void* state_workspace, uint64_t state_bytes,
                       void* cuda_stream, uint64_t* digest) {
  WsLayout w;
  const int rc = state_check(sim, state_workspace, state_bytes, &w);
  if (rc != GORGO_OK) return rc;
  if (!digest) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  unsigned char* base = static_cast<unsigned char*>(state_workspace);
  DigestArgs d = {};
  d.m = sim->m; d.tr = sim->tr; d.states = base + w.states; d.lay = w.st;
  d.route_log = base + w.route_log; d.route_log_stride = sim->tr.n_req;
  d.digest = digest;
  if (launch_digest(d, 1, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return GORGO_ERR_CUDA;
  return GORGO_OK;
}

int gorgo_state_status(gorgo_sim_t* sim, void* state_workspace, uint64_t state_bytes,
                       void* cuda_stream, uint64_t* requests_seen) {
  WsLayout w;
  const int rc = state_check(sim, state_workspace, state_bytes, &w);
  if (rc != GORGO_OK) return rc;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CandHeader h;
  if (cudaMemcpyAsync(&h, static_cast<unsigned char*>(state_workspace) + w.states, sizeof(h),
                      cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return GORGO_ERR_CUDA;
  if (requests_seen) *requests_seen = h.processed;
  return h.status;
}

int gorgo_replay_occupancy(gorgo_sim_t* sim, int32_t* ctas_per_sm, uint64_t* smem_bytes_per_cta) {
  if (!sim || !ctas_per_sm) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  const int n = replay_occupancy(sim->m, smem_bytes_per_cta);
  if (n < 0) return GORGO_ERR_CUDA;
  *ctas_per_sm = n;
  return GORGO_OK;
}

int gorgo_measure_gather(int device, void* buffer, uint64_t buffer_bytes, uint64_t footprint_bytes,
                         void* cuda_stream, double* sectors_gb_per_s) {
  if (!buffer || !sectors_gb_per_s || (uintptr_t)buffer % kAlign) return GORGO_ERR_INVALID_ARG;
  if (footprint_bytes < 4096 || footprint_bytes + 256 > buffer_bytes) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return GORGO_ERR_CUDA;
  const uint32_t blocks = (uint32_t)prop.multiProcessorCount * 8u;   // 2,048 threads per SM
  const uint32_t per_thread = 256;
  const uint64_t n_sectors = footprint_bytes / 32;
  uint32_t* sink = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(buffer) + footprint_bytes / 256 * 256);
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess) return GORGO_ERR_CUDA;
  if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return GORGO_ERR_CUDA; }
  int rc = GORGO_OK;
  float best_ms = 0.f;
  for (int rep = 0; rep < 4 && rc == GORGO_OK; ++rep) {        // first pass warms up
    if (cudaEventRecord(e0, st) != cudaSuccess ||
        launch_gather(buffer, n_sectors, per_thread, blocks, sink, st) != cudaSuccess ||
        cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) {
      rc = GORGO_ERR_CUDA;
      break;
    }
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = GORGO_ERR_CUDA; break; }
    if (rep > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (rc != GORGO_OK) { cudaGetLastError(); return rc; }
  const double sectors = (double)blocks * 256.0 * per_thread;
  *sectors_gb_per_s = sectors * 32.0 / (best_ms * 1e-3) / 1e9;
  return GORGO_OK;
}

int gorgo_debug_set(gorgo_sim_t* sim, uint32_t what, uint32_t value) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  switch (what) {
    case GORGO_DEBUG_POLL_LIMIT: sim->poll_limit = value; break;
    case GORGO_DEBUG_RING_POLLS: sim->ring_polls = value; break;
    case GORGO_DEBUG_PROBE_OFF: sim->probe_off = value ? 1u : 0u; break;
    case GORGO_DEBUG_SCOUT_OFF: sim->scout_off = value ? 1u : 0u; break;
    default: return GORGO_ERR_INVALID_ARG;
  }
  return GORGO_OK;
}

int gorgo_set_profiling(gorgo_sim_t* sim, int enable) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  if (enable && sim->ev.empty()) {
    DeviceGuard guard(sim->device);
    if (!guard.ok) return GORGO_ERR_CUDA;
    sim->ev.resize(64);
    for (size_t i = 0; i < sim->ev.size(); ++i) {
      if (cudaEventCreate(&sim->ev[i]) != cudaSuccess) {
        for (size_t j = 0; j < i; ++j) cudaEventDestroy(sim->ev[j]);
        sim->ev.clear();
        return GORGO_ERR_CUDA;
      }
    }
  }
  if (enable && sim->wev.empty()) {
    DeviceGuard guard(sim->device);
    if (!guard.ok) return GORGO_ERR_CUDA;
    sim->wev.resize(64);
    for (size_t i = 0; i < sim->wev.size(); ++i) {
      if (cudaEventCreate(&sim->wev[i]) != cudaSuccess) {
        for (size_t j = 0; j < i; ++j) cudaEventDestroy(sim->wev[j]);
        sim->wev.clear();
        return GORGO_ERR_CUDA;
      }
    }
  }
  sim->profiling = enable != 0;
  sim->ev_used = 0;
  sim->wev_used = 0;
  return GORGO_OK;
}

int gorgo_last_window_ms(gorgo_sim_t* sim, double* window_ms, uint32_t* launches) {
  if (!sim || !window_ms) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  double sum = 0.0;
  for (uint32_t i = 0; i + 1 < sim->wev_used; i += 2) {
    float ms = 0.f;
    if (cudaEventSynchronize(sim->wev[i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, sim->wev[i], sim->wev[i + 1]) != cudaSuccess)
      return GORGO_ERR_CUDA;
    sum += ms;
  }
  *window_ms = sum;
  if (launches) *launches = sim->wev_used / 2;
  return GORGO_OK;
}

int gorgo_last_replay_ms(gorgo_sim_t* sim, double* replay_ms, uint32_t* launches) {
  if (!sim || !replay_ms) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(sim->device);
  if (!guard.ok) return GORGO_ERR_CUDA;
  double sum = 0.0;
  for (uint32_t i = 0; i + 1 < sim->ev_used; i += 2) {
    float ms = 0.f;
    if (cudaEventSynchronize(sim->ev[i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, sim->ev[i], sim->ev[i + 1]) != cudaSuccess)
      return GORGO_ERR_CUDA;
    sum += ms;
  }
  *replay_ms = sum;
  if (launches) *launches = sim->ev_used / 2;
  return GORGO_OK;
}

// ---- evaluation without any caller- or library-side allocation ---------------------------
// Scratch that ships with the library image: every GPU that loads libgorgo_b200 reserves this
// much global memory until the process exits.  In host code `g_static_scratch` is only a handle
// for the runtime, not an address a kernel could use; the device address is looked up once per
// device with cudaGetSymbolAddress (that device being current) and kept here.
static __device__ __align__(256) unsigned char g_static_scratch[GORGO_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on the CURRENT device (looked up on first use).
int static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return GORGO_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[device]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return GORGO_ERR_CUDA;
    }
    g_scratch_ptr[device] = p;
  }
  *out = g_scratch_ptr[device];
  return GORGO_OK;
}
}  // namespace

int gorgo_eval_population_static(gorgo_sim_t* sim, uint32_t n_candidates, const double* params,
                                 double time_scale, void* cuda_stream, double* p95_ttft_ms,
                                 double* p95_e2e_ms, uint8_t* route, uint16_t* hit_blocks,
                                 int32_t* cand_status) {
  if (!sim) return GORGO_ERR_INVALID_ARG;
  if (!sim->has_trace) return GORGO_ERR_NO_TRACE;
  // one candidate's replay state must fit; a larger population then runs in waves inside it
  if (make_ws(sim, 1, true).total > (uint64_t)GORGO_STATIC_SCRATCH_BYTES)
    return GORGO_ERR_STATIC_LIMIT;
  void* scratch = nullptr;
  {
    DeviceGuard guard(sim->device);
    if (!guard.ok) return GORGO_ERR_CUDA;
    const int rc = static_scratch_address(sim->device, &scratch);
    if (rc != GORGO_OK) return rc;
  }
  // the evaluation clears the cache masks and replica/slot state of every wave before replaying,
  // so whatever an earlier call left in the array is never read
  return eval_impl(sim, n_candidates, params, time_scale, scratch, GORGO_STATIC_SCRATCH_BYTES,
                   static_cast<cudaStream_t>(cuda_stream), p95_ttft_ms, p95_e2e_ms, route,
                   hit_blocks, nullptr, nullptr, cand_status, false);
}

#ifdef GORGO_PROF
// Cycle-accounting build only (not declared in gorgo.h, not part of the product library):
// waits for the device, copies the 64 phase accumulators out and clears them.
int gorgo_debug_phase_cycles(gorgo_sim_t* sim, uint64_t* out64) {
  if (!sim || !out64) return GORGO_ERR_INVALID_ARG;
  DeviceGuard guard(sim->device);
  if (!guard.ok || cudaDeviceSynchronize() != cudaSuccess) return GORGO_ERR_CUDA;
  return prof_read(reinterpret_cast<unsigned long long*>(out64), true) == cudaSuccess
             ? GORGO_OK : GORGO_ERR_CUDA;
}
#endif

const char* gorgo_strerror(int code) {
  switch (code) {
    case GORGO_OK: return "ok";
    case GORGO_ERR_INVALID_ARG: return "invalid argument";
    case GORGO_ERR_BAD_TRACE: return "trace violates a precondition";
    case GORGO_ERR_NONFINITE_PARAM: return "non-finite parameter or time scale";
    case GORGO_ERR_WORKSPACE_TOO_SMALL: return "device buffer too small";
    case GORGO_ERR_CUDA: return "CUDA runtime error";
    case GORGO_ERR_DEVICE_LIMIT: return "device-side loop limit reached";
    case GORGO_ERR_NO_TRACE: return "no trace uploaded";
    case GORGO_ERR_OUT_OF_ORDER: return "request batch out of order";
    case GORGO_ERR_STATIC_LIMIT: return "problem does not fit the library's built-in scratch array";
    default: return "unknown gorgo status";
  }
}

}  // extern "C"

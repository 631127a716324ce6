// Kernels of libgorgo_b200 (sm_100a): population replay, p95 selection, state digest, reset.
//
// Data layout chosen for this machine rather than per-replica hash tables:
//  * block ids are dense 32-bit numbers (renumbered at upload in order of first appearance, so
//    the blocks of one conversation are runs of consecutive numbers);
//  * per candidate ONE direct-indexed array `mask[id]` whose bit i says "block id is cached on
//    replica i".  A request's prefix probe on all R replicas is one coalesced read of its n
//    mask words and one ballot per replica that holds its first block;
//  * exact LRU without per-block recency stamps: the recency order of replica i is the order of
//    the requests routed to it (a linked list through `lru_next`), deepest block first inside a
//    request.  An eviction cursor walks that order; a touch (request n, position k) is still the
//    block's latest touch on replica i iff no later occurrence of the block (static
//    `occ_next` links computed at upload) belongs to a request routed to i.  Live touches at
//    the cursor are the LRU victims; stale ones are skipped for good;
//  * completions as per-request lists: a routed request stops counting in the queue signal at
//    the first later request that arrives at or after its finish time; the service warp finds
//    that request (time grid over the arrivals, then a 32-wide window) and pushes the completion
//    onto its list, the expiry warp sums every request's list ahead of the route warp.
// Requests are strictly ordered inside a candidate and every step depends on the one before, so
// a replay is bound by the latency of that chain, not by bandwidth.  One CTA of twelve warps
// replays one candidate and the warps split the chain:
//   route    queue signal, score (Eq. 3), argmin; reads no global memory;
//   gate     decides whether the staged prefix hits of the next request may be used, else
//            waits for the commits concerned and probes itself; posts the commit jobs;
//   probe    (two warps) run up to kWindow requests ahead: read block ids and mask words,
//            probe them and stage hits and the hit-dependent part of the score;
//   commit   (three warps, replicas split) size and perform the eviction, set the mask bits,
//            keep the recency lists;
//   scout    (two warps) validate touches ahead of every replica's eviction cursor and keep a
//            ring of ready victims per replica;
//   service  slots, start / first-token / finish times, outputs, completion filing;
//   expiry   completion sums per request.
// A staged read may predate the commits of the last kWindow requests; the gate warp knows which
// of those commits can have touched the request (shared block, or evicted block that occurs in
// it) and then repeats the read itself, so results never depend on the timing of the warps.
#include "gorgo_internal.h"

namespace gorgo {

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;

// Cycle accounting of the warps (built only with -DGORGO_PROF; the normal library
// carries none of it).  Every lap adds the SM clock ticks since the previous lap of the same
// warp to one of 16 per-role accumulators; the totals of all candidates end up in g_prof.
#ifdef GORGO_PROF
__device__ unsigned long long g_prof[64];
#define PROF_BEGIN() unsigned long long pf[16] = {}; long long pf_t = clock64()
#define PROF_LAP(k) do { const long long pf_n = clock64(); pf[k] += (unsigned long long)(pf_n - pf_t); pf_t = pf_n; } while (0)
#define PROF_ADD(k, v) pf[k] += (unsigned long long)(v)
#define PROF_END(base) do { if (lane == 0) { _Pragma("unroll") for (int pf_i = 0; pf_i < 16; ++pf_i) atomicAdd(&g_prof[(base) + pf_i], pf[pf_i]); } } while (0)
#else
#define PROF_BEGIN() do {} while (0)
#define PROF_LAP(k) do {} while (0)
#define PROF_ADD(k, v) do {} while (0)
#define PROF_END(base) do {} while (0)
#endif

__device__ __forceinline__ double d_inf() { return __longlong_as_double(0x7FF0000000000000LL); }

template <typename T> struct MaskOps;
template <> struct MaskOps<uint8_t>  { using Sh = uint32_t; };
template <> struct MaskOps<uint16_t> { using Sh = uint32_t; };
template <> struct MaskOps<uint32_t> { using Sh = uint32_t; };
template <> struct MaskOps<uint64_t> { using Sh = uint64_t; };

template <typename MaskT>
__device__ __forceinline__ MaskT shfl_up_mask(MaskT v, int d) {
  using Sh = typename MaskOps<MaskT>::Sh;
  return (MaskT)__shfl_up_sync(kFull, (Sh)v, d);
}
template <typename MaskT>
__device__ __forceinline__ MaskT shfl_mask(MaskT v, int src) {
  using Sh = typename MaskOps<MaskT>::Sh;
  return (MaskT)__shfl_sync(kFull, (Sh)v, src);
}
template <typename MaskT>
__device__ __forceinline__ int first_bit(MaskT v) {  // v != 0
  if (sizeof(MaskT) == 8) return __ffsll((long long)v) - 1;
  return __ffs((int)(uint32_t)v) - 1;
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
  return v;
}
// Order-preserving 64-bit key of a double (no NaN): -0.0 is folded onto +0.0 first so that the
// two zeros tie, as they do under '<'.
__device__ __forceinline__ uint64_t order_key(double v) {
  const uint64_t b = (uint64_t)__double_as_longlong(__dadd_rn(v, 0.0));
  return (b >> 63) ? ~b : (b | 0x8000000000000000ULL);
}
// Warp-wide minimum of 64-bit keys with the lowest index among equal keys; lanes that do not
// take part pass key = ~0 and idx = kNone.  Returns the winning index, the key through `key`.
__device__ __forceinline__ uint32_t warp_argmin_key(uint64_t& key, uint32_t idx) {
  const uint32_t hi = (uint32_t)(key >> 32), lo = (uint32_t)key;
  const uint32_t mh = __reduce_min_sync(kFull, hi);
  const uint32_t ml = __reduce_min_sync(kFull, hi == mh ? lo : 0xFFFFFFFFu);
  const bool win = hi == mh && lo == ml;
  key = ((uint64_t)mh << 32) | ml;
  return __reduce_min_sync(kFull, win ? idx : kNone);
}

// Is the touch at flat position g (a block of a request routed to replica `rep`) no longer
// the block's latest touch there, looking at requests up to `r_now`?  `rep_now` is the route of
// request r_now if its log entry has not been written yet (else pass the logged value).
__device__ __forceinline__ bool touch_is_stale(const TraceView& tr, const uint8_t* route_log,
                                               uint32_t g, uint32_t rep, uint32_t r_now,
                                               uint32_t rep_now) {
  uint2 nx = tr.occ_next[g];
  #pragma unroll 1
  while (nx.x != kNone && nx.y <= r_now) {
    const uint32_t rt = (nx.y == r_now) ? rep_now : (uint32_t)route_log[nx.y];
    if (rt == rep) return true;
    nx = tr.occ_next[nx.x];
  }
  return false;
}

__device__ __forceinline__ uint64_t mix64(uint64_t z) {  // splitmix64 finaliser
  z ^= z >> 30; z *= 0xbf58476d1ce4e5b9ULL;
  z ^= z >> 27; z *= 0x94d049bb133111ebULL;
  z ^= z >> 31;
  return z;
}

// ------------------------------------------------------------------------------ replay

// Clear `bit` of mask[id] without reading it back (a reduction performed in L2).
template <typename MaskT>
__device__ __forceinline__ void mask_clear_bit(MaskT* mask, uint32_t id, MaskT bit) {
  if (sizeof(MaskT) == 8) {
    atomicAnd(reinterpret_cast<unsigned long long*>(mask) + id, ~(unsigned long long)bit);
  } else {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(mask + id);
    const uint32_t sh = (uint32_t)(addr & 3u) * 8u;
    atomicAnd(reinterpret_cast<unsigned int*>(addr & ~(uintptr_t)3), ~((uint32_t)bit << sh));
  }
}
// Set `bit` of mask[id] the same way.
template <typename MaskT>
__device__ __forceinline__ void mask_set_bit(MaskT* mask, uint32_t id, MaskT bit) {
  if (sizeof(MaskT) == 8) {
    atomicOr(reinterpret_cast<unsigned long long*>(mask) + id, (unsigned long long)bit);
  } else {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(mask + id);
    const uint32_t sh = (uint32_t)(addr & 3u) * 8u;
    atomicOr(reinterpret_cast<unsigned int*>(addr & ~(uintptr_t)3), (uint32_t)bit << sh);
  }
}
// Mask words are read around L1: they are changed by reductions in L2.
template <typename MaskT>
__device__ __forceinline__ MaskT mask_load(const MaskT* mask, uint32_t id) {
  return __ldcg(mask + id);
}
template <>
__device__ __forceinline__ uint8_t mask_load<uint8_t>(const uint8_t* mask, uint32_t id) {
  return __ldcg(reinterpret_cast<const unsigned char*>(mask) + id);
}
template <>
__device__ __forceinline__ uint16_t mask_load<uint16_t>(const uint16_t* mask, uint32_t id) {
  return __ldcg(reinterpret_cast<const unsigned short*>(mask) + id);
}
template <>
__device__ __forceinline__ uint64_t mask_load<uint64_t>(const uint64_t* mask, uint32_t id) {
  return __ldcg(reinterpret_cast<const unsigned long long*>(mask) + id);
}
constexpr int kRegChunks = 3;     // request blocks held in registers: 3 x 32 = 96
constexpr uint32_t kListCap = 256;     // pre-validated eviction victims kept per replica
constexpr uint32_t kScouts = 2;        // scout warps per candidate (replicas split between them)
constexpr int kScoutBatches = 1;       // touches examined per lane and scout round
constexpr uint32_t kPostMargin = 512;  // start pre-validating when a cache is this close to full

constexpr uint32_t kStageDepth = 14;                   // requests staged by the probe warps (> kWindow)
constexpr uint32_t kStageBlocks = kRegChunks * 32u;    // blocks of a request kept per stage
constexpr uint32_t kWindow = 12;  // a staged read may be up to this many commits old (<= 32)
constexpr uint32_t kProbes = 2;   // probe warps per candidate (requests alternate between them)

// rings and counts of the warps of one candidate
constexpr uint32_t kRouteRing = 32;   // routes handed from the route warp to the service warp
constexpr uint32_t kRouteLead = 24;   // the route warp runs at most this far ahead of the service warp
constexpr uint32_t kExpRing = 8;      // completion sums published ahead of the route warp
constexpr uint32_t kCommitWarps = 3;  // commit warps per candidate (replicas split between them)
constexpr uint32_t kJobRing = 32;     // routed requests handed from the gate warp to the commit warps
constexpr uint32_t kHitRing = 16;     // tags of requests hit by a recent eviction (> kWindow)
constexpr uint32_t kServices = 1;      // service warps per candidate (replicas split between them)

// Shared-memory view of one candidate's small state.
struct Smem {
  double* rtt; double* wrtt; double* w;
  long long* load;                // in-flight input tokens per replica (as of the last launch; the route warp keeps the live value)
  long long* cnt;                 // in-flight requests per replica (kept when the queue signal counts requests)
  uint32_t* occ; uint32_t* curreq; int32_t* curpos; uint32_t* lrutail;
  volatile uint32_t* progress;    // [kCommitWarps] requests each commit warp has passed
  volatile uint32_t* abort_flag;  // a bounded wait ran out: the other waits stop too
  volatile uint32_t* jobs;        // requests handed to the commit warps
  uint2* job;                     // [kJobRing] (replica | stage << 8 | blocks << 16, offset of the request's ids)
  // hand-over between the route, service and expiry warps
  volatile uint32_t* routed;      // requests routed so far
  volatile uint32_t* serviced;    // [kServices] requests each service warp has passed (serviced and filed, or not its own)
  volatile uint32_t* exp_ready;   // requests whose completion sums are published
  uint32_t* route_ring;           // [kRouteRing] chosen replica | prefix hit there << 8
  long long* exp_sum;             // [kExpRing][R] tokens (or requests) that completed by the request's arrival
  // eviction rings, one per replica: filled by the scout warp, drained by the commit warp.
  // entry = (block id, request of the block's next occurrence after the entry was made or kNone,
  //          position of the touch in its request, request of the touch), in eviction order
  uint4* lst;                     // [R][kListCap]
  volatile uint32_t* act;         // replay -> scout: the replica's cache is close to full
  volatile uint32_t* ring_head;   // entries consumed (commit warp)
  volatile uint32_t* ring_tail;   // entries produced (scout warp)
  volatile uint32_t* scan_cr;     // scout's own cursor into the recency order (set at activation)
  volatile int32_t* scan_cp;
};

// Requests committed on every replica: the slowest commit warp's position.
__device__ __forceinline__ uint32_t committed(const Smem& sm) {
  uint32_t v = sm.progress[0];
#pragma unroll
  for (uint32_t k = 1; k < kCommitWarps; ++k) v = min(v, sm.progress[k]);
  return v;
}
// Bounded wait until every request < want is committed.
__device__ __forceinline__ void wait_committed(const Smem& sm, uint32_t want, uint32_t limit, int32_t& status) {
  uint32_t polls = 0;
  while ((int32_t)(committed(sm) - want) < 0) {
    if (*sm.abort_flag) break;
    if (++polls > limit) { status = -6; *sm.abort_flag = 1; break; }
    __nanosleep(20);
  }
}

// Requests every service warp has passed.
__device__ __forceinline__ uint32_t serviced_all(const Smem& sm) {
  uint32_t v = sm.serviced[0];
#pragma unroll
  for (uint32_t k = 1; k < kServices; ++k) v = min(v, sm.serviced[k]);
  return v;
}
__device__ __forceinline__ uint32_t wait_serviced(const Smem& sm, uint32_t want, uint32_t limit, int32_t& status) {
  uint32_t polls = 0;
  uint32_t v = serviced_all(sm);
  while ((int32_t)(v - want) < 0) {
    if (*sm.abort_flag) break;
    if (++polls > limit) { status = -6; *sm.abort_flag = 1; break; }
    __nanosleep(20);
    v = serviced_all(sm);
  }
  return v;
}

// Scout warp: for every replica whose cache is close to full it walks the recency order ahead
// of the eviction cursor and appends to the replica's ring the touches that are still the latest
// touch of their block (the coming eviction victims, in order).  The commit warp evicts from the
// ring instead of validating touches on its critical path; entries that went stale after they
// were appended are recognised there by their next-occurrence field.
template <typename MaskT>
__device__ __forceinline__ void scout_warp(const ReplayArgs& a, const Smem& sm, const uint32_t* lru_next,
                           const uint8_t* route_log, uint32_t lane, uint32_t which) {
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  const uint32_t end = a.first + a.count;
  const uint32_t R = a.m.R;
  uint32_t idle = 0;
  uint32_t blocked0 = kNone - 1, blocked1 = kNone - 1;  // lru tail seen when the scan ran dry
  if (a.scout_off) return;                               // (test switch: the commit warps find their victims themselves)
  while (true) {
    const uint32_t prog = committed(sm);
    if (prog >= end || *sm.abort_flag) break;
    // the active replica with the emptiest ring that can still be extended
    uint32_t best = kNone;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const uint32_t i = lane + 32u * half;
      if (i < R && (i % kScouts) == which && sm.act[i]) {
        const uint32_t fill = sm.ring_tail[i] - sm.ring_head[i];
        const uint32_t bl = half ? blocked1 : blocked0;
        if (fill + 32u * kScoutBatches <= kListCap && sm.lrutail[i] != bl)
          best = min(best, (fill << 8) | i);
      }
    }
    best = __reduce_min_sync(kFull, best);
    if (best == kNone || prog == a.first) {
      if (++idle > (1u << 26)) break;              // bounded wait
      __nanosleep(64);
      continue;
    }
    idle = 0;
    const uint32_t i = best & 255u;
    __threadfence_block();
    const uint32_t rs = prog - 1;                  // every request <= rs is fully committed
    uint32_t cr = sm.scan_cr[i];
    int32_t cp = sm.scan_cp[i];
    uint32_t coff = (cr != kNone) ? req[cr].off : 0u;
    uint32_t tail = sm.ring_tail[i];
    uint4* out = sm.lst + (size_t)i * kListCap;
    bool dry = false;
    #pragma unroll 1
    for (uint32_t round = 0; round < 6; ++round) {
      const uint32_t room = kListCap - (tail - sm.ring_head[i]);
      if (room < 32u * kScoutBatches) break;
      if (cp < 0) {
        const uint32_t nx = (cr == kNone) ? kNone : __ldcg(lru_next + cr);
        if (nx == kNone || nx > rs) { dry = true; break; }   // end of the order as of rs
        cr = nx;
        const ReqRec cre = req[cr];
        coff = cre.off;
        cp = (int32_t)cre.nblk - 1;
        continue;
      }
      // kScoutBatches x 32 touches, deepest position first; issue every first load up front
      int32_t k[kScoutBatches];
      uint32_t id[kScoutBatches];
      uint2 c[kScoutBatches];
#pragma unroll
      for (int u = 0; u < kScoutBatches; ++u) {
        k[u] = cp - (int32_t)(u * 32u + lane);
        id[u] = 0;
        c[u] = make_uint2(kNone, kNone);
        if (k[u] >= 0) {
          const uint32_t g = coff + (uint32_t)k[u];
          id[u] = ids[g];
          c[u] = a.tr.occ_next[g];
        }
      }
#pragma unroll
      for (int u = 0; u < kScoutBatches; ++u) {
        bool live = k[u] >= 0;
        uint32_t nxr = kNone;
        if (live) {
          uint2 cc = c[u];
          #pragma unroll 1
          while (cc.x != kNone && cc.y <= rs) {       // later occurrences up to rs
            if ((uint32_t)__ldcg(route_log + cc.y) == i) { live = false; break; }
            cc = a.tr.occ_next[cc.x];
          }
          if (live && cc.x != kNone) nxr = cc.y;      // first occurrence after rs
        }
        const unsigned lv = __ballot_sync(kFull, live);
        const uint32_t slot = tail + (uint32_t)__popc(lv & ((1u << lane) - 1u));
        if (live) out[slot % kListCap] = make_uint4(id[u], nxr, (uint32_t)k[u], cr);
        tail += __popc(lv);
      }
      cp -= 32 * kScoutBatches;
      // every lane's entries are stored before lane 0 publishes the new tail (the lanes that
      // listed nothing must not run ahead of the ones that did)
      __syncwarp();
      __threadfence_block();
      if (lane == 0) {
        sm.scan_cr[i] = cr;
        sm.scan_cp[i] = cp;
        sm.ring_tail[i] = tail;
      }
    }
    if (dry) {
      const uint32_t lt = sm.lrutail[i];
      if ((i & 31u) == lane) { if (i < 32) blocked0 = lt; else blocked1 = lt; }
    }
    __syncwarp();
  }
}

// Holds the compiler back where shared-memory data is handed from one warp to another through a
// flag: a warp's shared-memory accesses are performed in program order, and a hardware fence
// would also wait for the warp's global loads in flight, which the pipelines below avoid.
__device__ __forceinline__ void smem_order() { asm volatile("" ::: "memory"); }

// Named CTA barriers pairing the route warp and the gate warp (32 + 32 threads each).  The
// barrier itself orders the arriving warp's earlier memory accesses before the waiting warp's
// later ones.
__device__ __forceinline__ void bar_arrive(int id) {
  asm volatile("bar.arrive %0, 64;" ::"r"(id) : "memory");
}
__device__ __forceinline__ void bar_wait(int id) {
  asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory");
}
constexpr int kBarHits = 1;    // gate warp -> route warp: prefix hits of the request are posted
constexpr int kBarRoute = 2;   // route warp -> gate warp: the chosen replica is posted

// Everything the warps of one candidate share.
template <typename MaskT>
struct Ctx {
  Smem sm;
  MaskT* mask;
  CandHeader* hdr;
  double* finish_log;
  uint32_t* exp_head;
  uint4* exp_rec;
  uint32_t* lru_next;
  uint8_t* route_log;
  double* free_at;             // [R*S] time each slot frees (shared or global memory)
  unsigned long long* slot_kv; // [R*S] KV tokens of each slot's newest request (global memory)
  volatile uint32_t* route;    // chosen replica of the current request
  volatile int32_t* status;    // first device-side limit hit by any warp
  // staging of the coming requests by the probe warp (kStageDepth stages + two of the gate warp)
  volatile uint32_t* st_ready; // [kStageDepth] request (+1) whose data the stage holds
  volatile uint32_t* probe_gone;  // the probe warp has stopped
  // (stages kStageDepth and kStageDepth+1 belong to the gate warp, used alternately)
  uint32_t* st_hits;           // [kStageDepth+2][R] prefix hit | blocks present << 16
  double* st_ab;               // [kStageDepth+2][R] (w_net*RTT + w_prefill*uncached) per replica
  uint4* st_meta;              // [kStageDepth+2] (input tokens, blocks | origin << 16, latest earlier request sharing a block, offset of its ids)
  unsigned long long* st_where;  // [kStageDepth+2] replicas that held any block of the request when it was read
  volatile uint32_t* evhit;    // [kHitRing] evhit[q % kHitRing] == q: a recent eviction took a block of request q
  uint32_t* st_ids;            // [kStageDepth+2][kStageBlocks] block ids
  MaskT* st_mk;                // [kStageDepth+2][kStageBlocks] mask words
  volatile uint32_t* hit_slot; // stage that holds the current request's hits and scores
};

// Bounded wait of one warp for a counter another warp of the candidate advances: polls until
// (int)(counter - want) >= 0.  If the limit runs out (or another warp already gave up) the
// candidate is marked failed and every later wait returns at once, so the CTA still terminates.
__device__ __forceinline__ uint32_t wait_counter(volatile uint32_t* counter, uint32_t want,
                                                 volatile uint32_t* abort_flag, uint32_t limit,
                                                 int32_t& status) {
  uint32_t v = *counter;
  uint32_t polls = 0;
  while ((int32_t)(v - want) < 0) {
    if (*abort_flag) break;
    if (++polls > limit) { status = -6; *abort_flag = 1; break; }
    __nanosleep(20);
    v = *counter;
  }
  return v;
}

// Epoch of the (scaled) time t under a time-varying network: the largest k in [0, n_epochs-1]
// with k * epoch_ms <= t (a quotient as first guess, then the defining comparison).
__device__ __forceinline__ uint32_t epoch_of(const ReplayArgs& a, double t) {
  const double q = t / a.epoch_ms;
  uint32_t k = q >= (double)(a.n_epochs - 1) ? a.n_epochs - 1 : (uint32_t)q;
  #pragma unroll 1
  while (k + 1 < a.n_epochs && __dmul_rn((double)(k + 1), a.epoch_ms) <= t) ++k;
  #pragma unroll 1
  while (k > 0 && __dmul_rn((double)k, a.epoch_ms) > t) --k;
  return k;
}

// Route warp: the serial chain of a replay.  Per request it adds the queue term to the staged
// part of the score of Eq. 3, takes the lowest-index argmin and posts the route.  Lane i (and
// i+32) keeps replica i's in-flight signal in registers: tokens (or requests) dispatched there,
// minus what the expiry warp reports as completed by this request's arrival.  The service model
// (slots, times) is not on this chain: it runs behind in the service warp.
// kBaseline compiles in the two switches of the paper's baseline policies (Section 4): a queue
// signal counted in requests, and routes fixed in advance; the plain cost-model replay is built
// without them.
template <typename MaskT, bool kBaseline>
__device__ __forceinline__ void route_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p, uint32_t lane) {
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R, K = a.m.K;
  const double w_que = sm.w[2];
  const bool by_requests = kBaseline && a.queue_in_requests != 0;   // baseline "least-request"
  int32_t status = 0;
  unsigned long long st_hit = 0, st_blk = 0;
  constexpr bool kWide = sizeof(MaskT) == 8;   // more than 32 replicas: two per lane
  const uint32_t i0 = lane, i1 = lane + 32u;
  long long ld0 = 0, ld1 = 0;          // in-flight signal of replicas lane and lane+32
  double nrm0 = 1.0, nrm1 = 1.0;       // their queue-load normalisers
  if (i0 < R) { ld0 = by_requests ? sm.cnt[i0] : sm.load[i0]; if (K != 3) nrm0 = sm.w[3 + i0]; }
  if (kWide && i1 < R) { ld1 = by_requests ? sm.cnt[i1] : sm.load[i1]; if (K != 3) nrm1 = sm.w[3 + i1]; }

  const uint32_t last_r = a.first + a.count - 1;
  // routes fixed in advance (baselines that do not look at the state), fetched two ahead
  const uint8_t* forced = kBaseline ? a.forced_route : nullptr;
  uint32_t fr_cur = forced ? forced[a.first] : 0u;
  uint32_t fr_nxt = forced ? forced[min(a.first + 1, last_r)] : 0u;
  uint32_t exp_seen = a.first, srv_seen = a.first;

  PROF_BEGIN();
  for (uint32_t j = 0; j < a.count; ++j) {
    const uint32_t r = a.first + j;

    // ---- completions the proxy has seen by this arrival (published by the expiry warp), and
    //      room in the ring of routes the service warp has not taken yet
    if ((int32_t)(exp_seen - (r + 1)) < 0)
      exp_seen = wait_counter(sm.exp_ready, r + 1, sm.abort_flag, a.poll_limit, status);
    if (r - srv_seen >= kRouteLead)
      srv_seen = wait_serviced(sm, r + 1 - kRouteLead, a.poll_limit, status);
    smem_order();
    PROF_LAP(0);
    const long long* gone = sm.exp_sum + (size_t)(r % kExpRing) * R;
    if (i0 < R) ld0 -= gone[i0];
    if (kWide && i1 < R) ld1 -= gone[i1];

    // ---- the queue part of the score does not need the prefix hits
    double cq0 = 0.0, cq1 = 0.0;
    if (i0 < R) { double q = (double)ld0; if (K != 3) q = __dmul_rn(q, nrm0); cq0 = __dmul_rn(w_que, q); }
    if (kWide && i1 < R) { double q = (double)ld1; if (K != 3) q = __dmul_rn(q, nrm1); cq1 = __dmul_rn(w_que, q); }
    PROF_LAP(1);

    bar_wait(kBarHits);                                   // prefix hits of request r are posted
    PROF_LAP(2);

    // ---- score of Eq. 3 (fixed order, no FMA): the staged (w_net*RTT + w_prefill*uncached)
    //      plus the queue term; lowest-index argmin
    const uint32_t stage = *cx.hit_slot;
    const uint4 meta = cx.st_meta[stage];                 // (this warp reads no global memory in its loop)
    const uint32_t in_tok = meta.x, n = meta.y & 0xFFFFu;
    uint64_t best_k = ~0ull;
    uint32_t best_i = kNone;
#pragma unroll
    for (int half = 0; half < (kWide ? 2 : 1); ++half) {
      const uint32_t i = lane + 32u * half;
      if (i < R) {
        double c = __dadd_rn(cx.st_ab[stage * R + i], half ? cq1 : cq0);
        if (c != c) c = (i == 0) ? -d_inf() : d_inf();  // a NaN score wins only at index 0
        const uint64_t ck = order_key(c);
        if (ck < best_k || best_i == kNone) { best_k = ck; best_i = i; }
      }
    }
    PROF_LAP(3);
    uint32_t istar = warp_argmin_key(best_k, best_i);
    if (kBaseline && forced) {
      istar = fr_cur;
      fr_cur = fr_nxt;
      fr_nxt = forced[min(r + 2, last_r)];
    }
    PROF_LAP(4);
    const uint32_t hstar = cx.st_hits[stage * R + istar] & 0xFFFFu;   // read before the stage can be reused
    if (lane == 0) {
      *cx.route = istar;
      cx.route_log[r] = (uint8_t)istar;
      sm.route_ring[r % kRouteRing] = istar | (hstar << 8);
      smem_order();
      *sm.routed = r + 1;
    }
    bar_arrive(kBarRoute);                                // the gate warp posts the commit of request r
    PROF_LAP(5);
    const long long add = by_requests ? 1ll : (long long)in_tok;
    if (istar == i0) ld0 += add;
    if (kWide && istar == i1) ld1 += add;
    st_hit += hstar; st_blk += n;
  }
  PROF_END(0);
  // the signal as of the last request routed
  if (i0 < R) { if (by_requests) sm.cnt[i0] = ld0; else sm.load[i0] = ld0; }
  if (kWide && i1 < R) { if (by_requests) sm.cnt[i1] = ld1; else sm.load[i1] = ld1; }
  status = __reduce_min_sync(kFull, status);
  if (lane == 0) {
    if (status != 0) atomicMin(const_cast<int32_t*>(cx.status), status);
    if (a.stats) {
      unsigned long long* s4 = reinterpret_cast<unsigned long long*>(a.stats) + (size_t)p * 4;
      atomicAdd(s4 + 1, st_hit);
      atomicAdd(s4 + 2, st_blk);
    }
  }
}

// First request x in [lo, hi] whose scaled arrival time is >= f; the caller knows that request
// hi qualifies.  Every lane walks the same bisection (broadcast loads).
__device__ __forceinline__ uint32_t first_arrival_at_or_after(const double* ts, double scale, double f,
                                                              uint32_t lo, uint32_t hi) {
  #pragma unroll 1
  while (lo < hi) {                                       // at most 32 rounds
    const uint32_t mid = lo + ((hi - lo) >> 1);
    if (__dmul_rn(scale, ts[mid]) >= f) hi = mid; else lo = mid + 1;
  }
  return lo;
}

// Service warp: the service model of a routed request (paper Eq. 1: network, queue wait,
// prefill), a few requests behind the route warp.  It takes the slot of the chosen replica that
// frees first, computes start, first-token and finish times, writes the outputs, and files the
// request under the first later request x that arrives at or after its finish time: that is
// when the proxy has seen its completion event, i.e. when it stops counting as in flight
// (signal of Eq. 2).  The search for x (a time grid over the arrivals, then a 32-wide window)
// and the list insertion need three dependent memory round trips; they run as a three-stage
// pipeline over consecutive requests so that none of them is waited for.
template <typename MaskT, bool kBaseline>
__device__ __forceinline__ void service_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p, uint32_t lane,
                                             uint32_t which) {
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R, S = a.m.S;
  const uint32_t N = a.tr.n_req;
  const ReqRec* req = a.tr.req;
  double* free_at = cx.free_at;
  const double scale = a.scales ? a.scales[p] : a.scale;   // time scale of this candidate
  const uint32_t end = a.first + a.count;
  const double t_last = __dmul_rn(scale, a.tr.ts[N - 1]);
  // grid bucket of a time: (time / scale) / grid_dt, as one multiplication; the search starts one
  // bucket early, which covers the rounding of this product many times over
  const bool use_grid = a.tr.grid_n > 0 && scale * a.tr.grid_dt >= 1e-280;
  const double to_bucket = use_grid ? 1.0 / (scale * a.tr.grid_dt) : 0.0;
  int32_t status = 0;

  // pipeline registers (uniform over the warp unless noted)
  uint32_t j1 = kNone, lo1 = 0, g1 = 0, tok1 = 0, rep1 = 0;  double f1 = 0.0;   // grid entry in flight (g1: lane 0)
  uint32_t j2 = kNone, lo2 = 0, tok2 = 0, rep2 = 0;  double f2 = 0.0, win2 = 0.0;   // window in flight (win2: per lane)
  uint32_t j3 = kNone, tok3 = 0, rep3 = 0, old3 = kNone;                       // list head exchange in flight (old3: lane 0)
  bool ins1 = false, ins2 = false, ins3 = false;   // the request gets a list entry (it completes before the trace ends)
  uint32_t s = a.first;
  uint32_t routed_seen = a.first, published = a.first;
  uint32_t idle = 0;
  bool failed = false;

  PROF_BEGIN();
  while (true) {
    // ---- what arrived since the last round
    const bool retired = j3 != kNone;
    if (retired && ins3 && lane == 0) cx.exp_rec[j3] = make_uint4(old3, tok3, rep3, 0u);
    uint32_t x2 = kNone;
    if (j2 != kNone && ins2) {
      const bool ok = lo2 + lane < N && __dmul_rn(scale, win2) >= f2;
      const unsigned b = __ballot_sync(kFull, ok);
      if (b) x2 = lo2 + (uint32_t)__ffs((int)b) - 1u;
      else x2 = first_arrival_at_or_after(a.tr.ts, scale, f2, min(lo2 + 32u, N - 1), N - 1);
    }
    const uint32_t g = __shfl_sync(kFull, g1, 0);
    PROF_LAP(0);
    // ---- publish how far this warp has got: every request before the oldest one it still works
    //      on is filed, or belongs to the other service warp
    {
      const uint32_t upto = j2 != kNone ? j2 : j1 != kNone ? j1 : s;
      if (upto != published) {
        published = upto;
        if (lane == 0) {
          if (retired) __threadfence_block();
          sm.serviced[which] = upto;
        }
      }
      if (upto == end) break;
    }
    PROF_LAP(1);
    // ---- next stage of each request in the pipeline
    j3 = j2; tok3 = tok2; rep3 = rep2; ins3 = ins2;
    if (j3 != kNone && ins3 && lane == 0) old3 = atomicExch(cx.exp_head + x2, j3);
    j2 = j1; tok2 = tok1; rep2 = rep1; f2 = f1; ins2 = ins1;
    if (j2 != kNone && ins2) {
      lo2 = max(lo1, use_grid ? g : 0u);
      win2 = lo2 + lane < N ? a.tr.ts[lo2 + lane] : 0.0;
    }
    j1 = kNone; ins1 = false;
    PROF_LAP(2);

    // ---- service model of the next routed request of this warp's replicas, if there is one
    if (s < end && (int32_t)(routed_seen - (s + 1)) < 0) routed_seen = *sm.routed;
    smem_order();
    #pragma unroll 1
    while (s < end && (int32_t)(routed_seen - (s + 1)) >= 0 &&
           (sm.route_ring[s % kRouteRing] & 0xFFu) % kServices != which) ++s;   // the other warp's
    if (s < end) {
      if ((int32_t)(routed_seen - (s + 1)) >= 0) {
        idle = 0;
        const ReqRec rec = req[s];
        const uint32_t rq = sm.route_ring[s % kRouteRing];
        const uint32_t istar = rq & 0xFFu, hstar = rq >> 8;
        const double t = __dmul_rn(scale, rec.ts_ms);
        const uint32_t in_tok = rec.in_tok;
        const unsigned long long hb = (unsigned long long)hstar * a.m.B;
        const uint32_t unc = in_tok - (uint32_t)(hb < in_tok ? hb : in_tok);
        // earliest-free slot, lowest index on ties (times are >= 0: bit patterns order like values)
        uint64_t bk = ~0ull;
        uint32_t bs = kNone;
        const double* fa = free_at + (size_t)istar * S;
        if (S <= 32) {
          if (lane < S) { bk = (uint64_t)__double_as_longlong(fa[lane]); bs = lane; }
        } else {
          #pragma unroll 1
          for (uint32_t s2 = lane; s2 < S; s2 += 32) {
            const uint64_t vk = (uint64_t)__double_as_longlong(fa[s2]);
            if (vk < bk || bs == kNone) { bk = vk; bs = s2; }
          }
        }
        bs = warp_argmin_key(bk, bs);
        PROF_LAP(3);
        const double bv = __longlong_as_double((long long)bk);   // the slot's free time
        double delay = sm.rtt[(size_t)rec.origin * R + istar];
        if (kBaseline && a.rtt_raw)        // time-varying network: the probe of the request's epoch
          delay = a.rtt_raw[((size_t)epoch_of(a, t) * a.m.G + rec.origin) * R + istar];
        const double arrive = __dadd_rn(t, delay);
        double start = (bv > arrive) ? bv : arrive;
        // (per-replica speeds and the extended service model only in the build that also carries
        // the baseline switches)
        const unsigned long long need_kv = (unsigned long long)in_tok + rec.out_tok;
        if (kBaseline && a.kv_budget > 0) {
          // admission under the KV budget: wait for other slots to finish until the request fits
          const unsigned long long* kv = cx.slot_kv + (size_t)istar * S;
          #pragma unroll 1
          for (uint32_t round = 0; round <= S; ++round) {
            unsigned long long usage = 0;
            uint64_t nf = ~0ull;                       // earliest finish among the other busy slots
            #pragma unroll 1
            for (uint32_t s2 = lane; s2 < S; s2 += 32) {
              const double f = fa[s2];
              if (s2 != bs && f > start) {
                usage += kv[s2];
                nf = min(nf, (uint64_t)__double_as_longlong(f));
              }
            }
            usage = warp_sum_u64(usage);
            uint32_t none = kNone;
            warp_argmin_key(nf, none);
            if (nf == ~0ull || usage + need_kv <= a.kv_budget) break;
            start = __longlong_as_double((long long)nf);
          }
        }
        const double pre_ms = (kBaseline && a.rep_prefill_ms) ? a.rep_prefill_ms[istar] : a.m.prefill_ms;
        double tok_ms = (kBaseline && a.rep_tpot_ms) ? a.rep_tpot_ms[istar] : a.m.tpot_ms;
        const double first = __dadd_rn(start, __dmul_rn(pre_ms, (double)unc));
        if (kBaseline && a.decode_slowdown > 0.0) {
          // a fuller batch decodes slower: busy slots at the first token, this one included
          uint32_t busy = 0;
          #pragma unroll 1
          for (uint32_t s2 = lane; s2 < S; s2 += 32) busy += (s2 != bs && fa[s2] > first) ? 1u : 0u;
          busy = __reduce_add_sync(kFull, busy);
          const double g = __dadd_rn(1.0, __dmul_rn(a.decode_slowdown, (double)busy));
          tok_ms = __dmul_rn(tok_ms, g);
        }
        const uint32_t dec_tok = rec.out_tok > 0 ? rec.out_tok - 1 : 0;
        const double finish = __dadd_rn(first, __dmul_rn(tok_ms, (double)dec_tok));
        if (lane == 0) {
          if (kBaseline && a.kv_budget > 0) cx.slot_kv[(size_t)istar * S + bs] = need_kv;
          free_at[(size_t)istar * S + bs] = finish;
          const size_t o = (size_t)p * a.out_stride + (s - a.first);
          if (a.route_out) a.route_out[o] = (uint8_t)istar;
          if (a.hit_out) a.hit_out[o] = (uint16_t)hstar;
          if (a.ttft_out) a.ttft_out[o] = __dsub_rn(first, t);
          if (a.e2e_out) a.e2e_out[o] = __dsub_rn(finish, t);
        }
        // the request stops counting at the first later arrival at or after `finish`
        j1 = s; f1 = finish; tok1 = in_tok; rep1 = istar;
        ins1 = s + 1 < N && t_last >= finish;
        lo1 = s + 1;
        if (!ins1 && cx.finish_log && lane == 0) {
          // completes after the last known arrival: chained in the state (read by the next launch)
          cx.finish_log[s] = finish;
          const uint32_t before = atomicExch(&cx.hdr->overflow, s + 1u);
          cx.exp_rec[s] = make_uint4(before - 1u, in_tok, istar, 0u);
        }
        if (ins1 && use_grid && lane == 0) {
          const double bf = __dmul_rn(finish, to_bucket);
          uint32_t b = 0;
          if (bf >= 2.0) b = (bf >= (double)a.tr.grid_n ? a.tr.grid_n : (uint32_t)bf) - 1u;
          g1 = a.tr.grid[b];
        }
        ++s;
        __syncwarp();
        PROF_LAP(4);
        continue;
      }
    }
    if (j2 == kNone && j3 == kNone && s < end) {   // nothing in flight and no route to take: wait
      if (*sm.abort_flag) failed = true;
      if (++idle > a.poll_limit) { status = -6; *sm.abort_flag = 1; failed = true; }
      if (failed) break;
      __nanosleep(40);
    }
    PROF_LAP(5);
  }
  PROF_END(16);
  status = __reduce_min_sync(kFull, status);
  if (lane == 0 && status != 0) atomicMin(const_cast<int32_t*>(cx.status), status);
}

// Expiry warp: for every request r, ahead of the route warp, the in-flight tokens (or requests)
// per replica whose completion the proxy has seen by r's arrival: the sum over r's list, filed by
// the service warp.  The list of r can only gain entries from requests j < r with finish <= t_r.
// finish_j >= t_j + tpot * decode tokens (network, waiting and prefill only add to it), so once
// every j < r whose bound lb_j = t_j + tpot*dec_j is <= t_r has been serviced, the list is
// final and is walked: one lane per request, eight requests in flight, one list hop per round.
template <bool kBaseline>
__device__ __forceinline__ void expiry_warp(const ReplayArgs& a, const Smem& sm, const uint32_t* exp_head,
                                            const uint4* exp_rec, volatile uint32_t* abort_flag,
                                            volatile int32_t* cta_status, uint32_t p, uint32_t lane) {
  const uint32_t R = a.m.R;
  const ReqRec* req = a.tr.req;
  const double scale = a.scales ? a.scales[p] : a.scale;
  const uint32_t end = a.first + a.count;
  const bool by_requests = kBaseline && a.queue_in_requests != 0;
  // smallest time per output token over the replicas (a lower bound of every decode time)
  double tok_ms = a.m.tpot_ms;
  if (kBaseline && a.rep_tpot_ms) {
    tok_ms = a.rep_tpot_ms[0];
    for (uint32_t i = 1; i < R; ++i) tok_ms = fmin(tok_ms, a.rep_tpot_ms[i]);
  }
  int32_t status = 0;
  double lb = d_inf();                 // bound of the latest request j with j % 32 == lane (none yet: +inf)
  uint32_t next_r = a.first;           // next request whose list walk starts
  uint32_t published = a.first;        // requests whose sums are published
  uint32_t my_r = kNone;               // lanes 0..7: request whose list this lane walks (kNone: idle)
  uint32_t e = kNone;                  //   entry whose record is in flight (kNone with my_r set: walk done)
  bool head_pending = false;           //   the list head is in flight
  uint32_t head_val = kNone;
  uint4 rec_val = make_uint4(kNone, 0u, 0u, 0u);
  uint32_t srv_seen = a.first, routed_seen = a.first;
  ReqRec rq_nxt = req[a.first];
  uint32_t idle = 0;

  while (published < end) {
    bool progress = false;
    // ---- what arrived: the head of a list, or one entry of it
    if (my_r != kNone) {
      if (head_pending) { e = head_val; head_pending = false; }
      else if (e != kNone) {
        long long* row = sm.exp_sum + (size_t)(my_r % kExpRing) * R;
        row[rec_val.z] += by_requests ? 1ll : (long long)rec_val.y;
        e = rec_val.x;
      }
    }
    // ---- publish finished walks in request order
    {
      const bool fin = my_r != kNone && !head_pending && e == kNone;
      unsigned m = __ballot_sync(kFull, fin) & 0xFFu;
      #pragma unroll 1
      while (m & (1u << (published % kExpRing))) {          // the lane of request `published` is done
        if (lane == published % kExpRing) my_r = kNone;
        m &= ~(1u << (published % kExpRing));
        ++published;
        progress = true;
      }
      if (progress && lane == 0) { smem_order(); *sm.exp_ready = published; }
    }
    // ---- start the walks of up to two more requests
    #pragma unroll 1
    for (int k = 0; k < 2 && next_r < end; ++k) {
      const uint32_t owner = next_r % kExpRing;
      // the ring row is free once the route warp has used its previous occupant
      if (next_r >= kExpRing + a.first && (int32_t)(routed_seen - (next_r - kExpRing + 1)) < 0) {
        routed_seen = *sm.routed;
        if ((int32_t)(routed_seen - (next_r - kExpRing + 1)) < 0) break;
      }
      if (__shfl_sync(kFull, my_r, owner) != kNone) break;    // its lane still walks (cannot happen once the row is free)
      const double t = __dmul_rn(scale, rq_nxt.ts_ms);
      // requests j in [next_r-32, next_r) whose completion may be visible at t: all up to the
      // latest of them must have been serviced
      const unsigned hz = __ballot_sync(kFull, lb <= t);
      const uint32_t rot = next_r & 31u;
      const unsigned in_order = __funnelshift_r(hz, hz, rot);   // bit k: request next_r - 32 + k
      const long long need = (long long)next_r - (long long)__clz((int)in_order);
      if ((long long)srv_seen < need) {
        srv_seen = serviced_all(sm);
        if ((long long)srv_seen < need) break;
      }
      __threadfence_block();   // the service warp's list stores before `serviced` are visible from here on
      // clear the row, start the walk
      long long* row = sm.exp_sum + (size_t)owner * R;
      if (lane < R) row[lane] = 0;
      if (lane + 32u < R) row[lane + 32u] = 0;
      __syncwarp();
      if (lane == owner) { my_r = next_r; head_pending = true; e = kNone; head_val = __ldcg(exp_head + next_r); }
      if (lane == rot) {
        const uint32_t dec_tok = rq_nxt.out_tok > 0 ? rq_nxt.out_tok - 1 : 0;
        lb = __dadd_rn(t, __dmul_rn(tok_ms, (double)dec_tok));
      }
      ++next_r;
      rq_nxt = req[min(next_r, end - 1)];
      progress = true;
    }
    // ---- next hop of every walk
    if (my_r != kNone && !head_pending && e != kNone) rec_val = __ldcg(exp_rec + e);
    if (progress) idle = 0;
    else {
      if (*abort_flag) break;
      if (++idle > a.poll_limit) { status = -6; *abort_flag = 1; break; }
      __nanosleep(40);
    }
  }
  status = __reduce_min_sync(kFull, status);
  if (lane == 0 && status != 0) atomicMin(const_cast<int32_t*>(cta_status), status);
}

// What a warp needs to know of a request ahead of time.
struct Ahead { uint32_t off, nblk, prev_share, in_tok, origin; double ts; };
__device__ __forceinline__ Ahead fetch_ahead(const ReqRec* req, uint32_t q, uint32_t end) {
  Ahead h = {0u, 0u, kNone, 0u, 0u, 0.0};
  if (q < end) {
    const ReqRec x = req[q];
    h.off = x.off; h.nblk = x.nblk; h.prev_share = x.prev_share; h.in_tok = x.in_tok;
    h.origin = x.origin; h.ts = x.ts_ms;
  }
  return h;
}

// Warp-wide OR of mask words.
template <typename MaskT>
__device__ __forceinline__ MaskT warp_or_mask(MaskT m) {
  if (sizeof(MaskT) == 8) {
    const uint32_t lo = __reduce_or_sync(kFull, (uint32_t)(uint64_t)m);
    const uint32_t hi = __reduce_or_sync(kFull, (uint32_t)((uint64_t)m >> 32));
    return (MaskT)(((uint64_t)hi << 32) | lo);
  }
  return (MaskT)__reduce_or_sync(kFull, (uint32_t)m);
}

// Probe of a request on every replica from staged mask words.  For this lane's replicas (lane
// and lane+32): h = leading blocks whose mask has the replica's bit (the prefix hit), p = all
// blocks of the request whose mask has it (what a commit there does not have to insert).  The
// first kStageBlocks words come from `smk`; longer prompts read the rest from memory.
template <typename MaskT, typename LoadWord>
__device__ __forceinline__ void probe_words(LoadWord load_word, uint32_t n, uint32_t R,
                                            uint32_t lane, uint32_t& h0, uint32_t& h1,
                                            uint32_t& p0, uint32_t& p1, unsigned long long& where) {
  h0 = 0; h1 = 0; p0 = 0; p1 = 0; where = 0;
  MaskT alive = (R >= sizeof(MaskT) * 8) ? (MaskT)~(MaskT)0 : (MaskT)((((MaskT)1) << (R & 63)) - 1);
  #pragma unroll 1
  for (uint32_t c = 0; c < n; c += 32) {
    const uint32_t k = c + lane;
    MaskT m = 0;
    if (k < n) m = load_word(c, k);
    MaskT it = warp_or_mask<MaskT>(m);      // replicas that hold any block of this chunk
    where |= (unsigned long long)it;
    MaskT still = 0;
    #pragma unroll 1
    while (it != 0) {
      const int i = first_bit<MaskT>(it);
      it &= (MaskT)(it - 1);
      const unsigned b = __ballot_sync(kFull, (m >> i) & 1);
      const uint32_t cnt = __popc(b);
      const bool running = (alive >> i) & 1;
      const uint32_t run = !running ? 0u : (b == kFull) ? 32u : (uint32_t)__ffs((int)~b) - 1u;
      if ((uint32_t)(i & 31) == lane) {
        if (sizeof(MaskT) != 8 || i < 32) { h0 += run; p0 += cnt; } else { h1 += run; p1 += cnt; }
      }
      if (run == 32u) still |= (MaskT)(((MaskT)1) << i);
    }
    alive = still;
  }
}

// The same from staged mask words: the first kStageBlocks words come from `smk`; longer prompts
// read the rest from memory.
template <typename MaskT>
__device__ __forceinline__ void probe_staged(const MaskT* smk, const MaskT* mask,
                                             const uint32_t* ids, const Ahead& q, uint32_t R,
                                             uint32_t lane, uint32_t& h0, uint32_t& h1,
                                             uint32_t& p0, uint32_t& p1, unsigned long long& where) {
  probe_words<MaskT>([&](uint32_t c, uint32_t k) -> MaskT {
    return (c < kStageBlocks) ? smk[k] : mask_load<MaskT>(mask, ids[q.off + k]);
  }, q.nblk, R, lane, h0, h1, p0, p1, where);
}

// Prefix hits of a request in the PROXY'S INDEX (extended build): bit i of a block's word says that
// an earlier request containing the block was routed to replica i, whatever the replica has
// evicted since.  The word is gathered by walking the block's earlier occurrences.
template <typename MaskT>
__device__ __forceinline__ void probe_index(const TraceView& tr, const uint8_t* route_log, const Ahead& q,
                                            uint32_t R, uint32_t lane, uint32_t& h0, uint32_t& h1) {
  uint32_t p0, p1;
  unsigned long long where;
  probe_words<MaskT>([&](uint32_t, uint32_t k) -> MaskT {
    unsigned long long w = 0;
    uint2 pv = tr.occ_prev[q.off + k];
    #pragma unroll 1
    for (uint32_t guard = 0; pv.x != kNone && guard < tr.n_req; ++guard) {
      w |= 1ull << ((uint32_t)__ldcg(route_log + pv.y) & 63u);
      pv = tr.occ_prev[pv.x];
    }
    return (MaskT)w;
  }, q.nblk, R, lane, h0, h1, p0, p1, where);
}

// Stage the prefix hits of a request and the part of its score (Eq. 3) that depends on them:
// ab_i = (w_net * RTT[g][i]) + (w_prefill * uncached_i), same operations and order as the score.
// st_hits packs (prefix hit, blocks present << 16) of a replica into one word.
template <typename MaskT, bool kBaseline>
__device__ __forceinline__ void stage_scores(const ReplayArgs& a, const Ctx<MaskT>& cx,
                                             const Ahead& q, uint32_t slot, uint32_t h0,
                                             uint32_t h1, uint32_t p0, uint32_t p1,
                                             unsigned long long where, uint32_t lane, double scale) {
  const uint32_t R = a.m.R;
  // (proxy index, extended build only: the score takes its hits from the index)
  uint32_t s0 = h0, s1 = h1;
  if (kBaseline && a.proxy_index) probe_index<MaskT>(a.tr, cx.route_log, q, R, lane, s0, s1);
  // (time-varying network, extended build only: the proxy's signal of the request's epoch)
  const double* ewma_row = nullptr;
  if (kBaseline && a.rtt_ewma)
    ewma_row = a.rtt_ewma + ((size_t)epoch_of(a, __dmul_rn(scale, q.ts)) * a.m.G + q.origin) * R;
  if (lane == 0) {
    cx.st_where[slot] = where;
    cx.st_meta[slot] = make_uint4(q.in_tok, q.nblk | (q.origin << 16), q.prev_share, q.off);
  }
  const double w_pre = cx.sm.w[1];
  const double* wrtt_row = cx.sm.wrtt + (size_t)q.origin * R;
#pragma unroll
  for (int half = 0; half < (sizeof(MaskT) == 8 ? 2 : 1); ++half) {
    const uint32_t i = lane + 32u * half;
    if (i < R) {
      const uint32_t h = half ? h1 : h0, pr = half ? p1 : p0;
      const unsigned long long hb = (unsigned long long)(half ? s1 : s0) * a.m.B;
      const uint32_t unc = q.in_tok - (uint32_t)(hb < q.in_tok ? hb : q.in_tok);
      cx.st_hits[slot * R + i] = h | (pr << 16);
      const double net = (kBaseline && ewma_row) ? __dmul_rn(cx.sm.w[0], ewma_row[i]) : wrtt_row[i];
      cx.st_ab[slot * R + i] = __dadd_rn(net, __dmul_rn(w_pre, (double)unc));
    }
  }
}

// Probe warp: runs up to kWindow requests ahead of the commit warps.  For request q it reads the
// block ids and the mask words (first kStageBlocks blocks), stages them in shared memory, probes
// them and publishes the prefix hits.  Its reads may predate the commits of the last kWindow
// requests; the gate warp knows which of those commits can have touched request q and then
// repeats the work itself, so this warp is an accelerator only and may stop at any time.
template <typename MaskT, bool kBaseline>
__device__ __forceinline__ void probe_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p,
                                           uint32_t lane, uint32_t which) {
  const double scale = a.scales ? a.scales[p] : a.scale;
  const Smem& sm = cx.sm;
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  const MaskT* mask = cx.mask;
  const uint32_t R = a.m.R;
  const uint32_t end = a.first + a.count;
  if (a.probe_off) { if (lane == 0) *cx.probe_gone = 1; return; }   // (test switch: the gate warp probes every request)
  const uint32_t q0 = a.first + which;                  // this warp takes requests q0, q0 + kProbes, ...
  Ahead q_a = fetch_ahead(req, q0, end), q_n = fetch_ahead(req, q0 + kProbes, end);
  Ahead q_b = q_a;
  uint32_t id_a[kRegChunks], id_n[kRegChunks], id_b[kRegChunks];
  MaskT m_a[kRegChunks], m_b[kRegChunks];
#pragma unroll
  for (int c = 0; c < kRegChunks; ++c) {
    const uint32_t k = c * 32u + lane;
    id_a[c] = (k < q_a.nblk) ? ids[q_a.off + k] : 0u;
    id_b[c] = 0u; m_b[c] = (MaskT)0;
  }
  for (uint32_t qa = q0; qa < end + kProbes; qa += kProbes) {
    if (qa < end) {
      // room: the stage of request qa is free and its read is at most kWindow commits old once
      // request qa - kWindow - 1 is committed, i.e. progress >= qa - kWindow
      uint32_t polls = 0;
      while ((int32_t)(committed(sm) - qa) < -(int32_t)kWindow) {
        if (++polls > (1u << 22) || *sm.abort_flag) { *cx.probe_gone = 1; return; }   // bounded wait
        __nanosleep(20);
      }
#pragma unroll
      for (int c = 0; c < kRegChunks; ++c) {
        const uint32_t k = c * 32u + lane;
        m_a[c] = (k < q_a.nblk) ? mask_load<MaskT>(mask, id_a[c]) : (MaskT)0;
        id_n[c] = (k < q_n.nblk) ? ids[q_n.off + k] : 0u;     // ids of the request after
      }
    }
    const Ahead q_nn = fetch_ahead(req, qa + 2 * kProbes, end);
    if (qa > q0) {
      // stage and probe this warp's previous request (its mask words were requested one round ago)
      const uint32_t qb = qa - kProbes, slot = qb % kStageDepth;
      uint32_t* sid = cx.st_ids + slot * kStageBlocks;
      MaskT* smk = cx.st_mk + slot * kStageBlocks;
#pragma unroll
      for (int c = 0; c < kRegChunks; ++c) {
        const uint32_t k = c * 32u + lane;
        if (k < q_b.nblk) { sid[k] = id_b[c]; smk[k] = m_b[c]; }
      }
      __syncwarp();
      uint32_t h0, h1, p0, p1;
      unsigned long long where;
      probe_staged<MaskT>(smk, mask, ids, q_b, R, lane, h0, h1, p0, p1, where);
      stage_scores<MaskT, kBaseline>(a, cx, q_b, slot, h0, h1, p0, p1, where, lane, scale);
      smem_order();
      __syncwarp();
      if (lane == 0) cx.st_ready[slot] = qb + 1;
    }
    q_b = q_a; q_a = q_n; q_n = q_nn;
#pragma unroll
    for (int c = 0; c < kRegChunks; ++c) { id_b[c] = id_a[c]; m_b[c] = m_a[c]; id_a[c] = id_n[c]; }
  }
}

// Gate warp: the partner of the route warp.  For every request it decides whether the prefix
// hits the probe warp staged are still exact, hands them to the route warp, and passes the routed
// request on to the commit warps.  A staged read of request q may predate the commits of the
// kWindow requests before q.  Such a commit can have changed q's hits only if it (a) shares a
// block with q -- known from the trace: `prev_share` -- or (b) evicted a block of q, which needs
// the commit to have been routed to a replica that held one of q's blocks when they were read
// (`st_where`).  If neither can be the case the staged hits go out the moment the previous route
// is known; otherwise the gate waits for the commits in question and looks at what they report
// (`evhit`), and if need be reads and probes the mask words again itself.
template <typename MaskT, bool kBaseline>
__device__ __forceinline__ void gate_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p,
                                          uint32_t lane) {
  const double scale = a.scales ? a.scales[p] : a.scale;
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R;
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  const MaskT* mask = cx.mask;
  int32_t status = 0;
  unsigned long long st_probe = 0;
  const uint32_t end = a.first + a.count;

  uint32_t my_req = kNone, my_rep = 0;   // lane l: the latest routed request with index % 32 == l, and its replica
  bool posted = false;             // the hits of the coming request were already handed over
  uint32_t slot = 0;               // stage that holds the current request's ids, mask words and hits
  // hand the hits of a request over to the route warp and count its probes
  auto hand_over = [&](uint32_t sl, uint32_t nblk) {
    if (lane == 0) *cx.hit_slot = sl;
    bar_arrive(kBarHits);                                 // the route warp may score the request
    if (a.stats) {                                        // probes the plain formula charges
      if (lane < R) { const uint32_t h = cx.st_hits[sl * R + lane] & 0xFFFFu; st_probe += (h + 1 < nblk ? h + 1 : nblk); }
      if (sizeof(MaskT) == 8 && lane + 32u < R) { const uint32_t h = cx.st_hits[sl * R + lane + 32u] & 0xFFFFu; st_probe += (h + 1 < nblk ? h + 1 : nblk); }
    }
  };
  // latest request among the kWindow before q that was routed to a replica in `where` (kNone: none)
  auto conflict = [&](uint32_t q, unsigned long long where) -> uint32_t {
    const bool hit = my_req != kNone && q - 1u - my_req < kWindow && ((where >> my_rep) & 1ull);
    if (!__any_sync(kFull, hit)) return kNone;
    return __reduce_max_sync(kFull, hit ? my_req : 0u);
  };
  // does a commit since its staged read share a block with request idx?  (prev: the latest earlier
  // request that shares a block with it)
  auto shares = [&](uint32_t prev, uint32_t idx) { return prev != kNone && prev + kWindow >= idx; };
  uint32_t n = 0, off_cur = 0;     // blocks of the current request, offset of its ids

  PROF_BEGIN();
  for (uint32_t r = a.first; r < end; ++r) {
    // ---- prefix hits of request r, unless they went out right after the previous route
    if (!posted) {
      const uint32_t ss = r % kStageDepth;
      bool staged = __shfl_sync(kFull, cx.st_ready[ss], 0) == r + 1;
      Ahead q_cur;
      if (staged) {
        smem_order();
        const uint4 meta = cx.st_meta[ss];
        q_cur.in_tok = meta.x; q_cur.nblk = meta.y & 0xFFFFu; q_cur.origin = meta.y >> 16;
        q_cur.prev_share = meta.z; q_cur.off = meta.w;
        q_cur.ts = (kBaseline && a.rtt_ewma) ? a.tr.ts[r] : 0.0;
      } else {
        q_cur = fetch_ahead(req, r, end);
      }
      n = q_cur.nblk; off_cur = q_cur.off;
      const bool sh = shares(q_cur.prev_share, r);
      uint32_t done_to = sh ? r : 0u;                         // requests < done_to must be committed
      if (!sh) {
        if (!staged && !*cx.probe_gone) {
          uint32_t polls = 0;
          while (cx.st_ready[ss] != r + 1 && !*cx.probe_gone && polls < 4096) { ++polls; __nanosleep(20); }
          // (one lane decides: every lane must take the same path)
          staged = __shfl_sync(kFull, cx.st_ready[ss], 0) == r + 1;
          smem_order();
        }
        if (staged) {
          const uint32_t c = conflict(r, cx.st_where[ss]);
          if (c != kNone) done_to = c + 1;
        }
      }
      if (!staged) done_to = r;
      PROF_LAP(3);
      if (done_to > a.first) wait_committed(sm, done_to, a.poll_limit, status);
      smem_order();
      PROF_LAP(4);
      if (!sh && staged && (done_to <= a.first || cx.evhit[r % kHitRing] != r)) {
        slot = ss;
      } else {
        // read and probe here, after every earlier request is committed
        PROF_ADD(11, 1);
        if (done_to < r) wait_committed(sm, r, a.poll_limit, status);
        uint32_t h0 = 0, h1 = 0, p0 = 0, p1 = 0;
        slot = kStageDepth + (r & 1u);                          // this warp's own stages
        uint32_t* sid = cx.st_ids + slot * kStageBlocks;
        MaskT* smk = cx.st_mk + slot * kStageBlocks;
        #pragma unroll 1
        for (uint32_t c = 0; c < n && c < kStageBlocks; c += 32) {
          const uint32_t k = c + lane;
          if (k < n) { const uint32_t id = ids[q_cur.off + k]; sid[k] = id; smk[k] = mask_load<MaskT>(mask, id); }
        }
        __syncwarp();
        unsigned long long where = 0;
        probe_staged<MaskT>(smk, mask, ids, q_cur, R, lane, h0, h1, p0, p1, where);
        stage_scores<MaskT, kBaseline>(a, cx, q_cur, slot, h0, h1, p0, p1, where, lane, scale);
        __syncwarp();
      }
      hand_over(slot, n);
    }
    PROF_LAP(0);

    bar_wait(kBarRoute);                                  // the replica has been chosen
    PROF_LAP(1);
    const uint32_t istar = *cx.route;
    if (lane == 0) {
      sm.job[r % kJobRing] = make_uint2(istar | (slot << 8) | (n << 16), off_cur);
      smem_order();
      *sm.jobs = r + 1;                                   // the commit warps may take request r
    }
    if (lane == (r & 31u)) { my_req = r; my_rep = istar; }

    // ---- the next request's hits go out now if no commit since their read can have touched them
    posted = false;
    if (r + 1 < end) {
      const uint32_t ss = (r + 1) % kStageDepth;
      if (__shfl_sync(kFull, cx.st_ready[ss], 0) == r + 2) {
        smem_order();
        const uint4 meta = cx.st_meta[ss];
        bool okk = !shares(meta.z, r + 1);
        if (okk) {
          // a commit routed to a holder of its blocks is no obstacle once it is done and did not
          // evict any of them
          const uint32_t c = conflict(r + 1, cx.st_where[ss]);
          if (c != kNone) okk = (int32_t)(committed(sm) - (c + 1)) >= 0 && cx.evhit[(r + 1) % kHitRing] != r + 1;
        }
        if (okk) {
          slot = ss;
          n = meta.y & 0xFFFFu; off_cur = meta.w;
          hand_over(slot, n);
          posted = true;
          PROF_ADD(14, 1);
        } else PROF_ADD(13, 1);
      } else PROF_ADD(12, 1);
    }
    PROF_LAP(2);
  }
  PROF_END(32);
  st_probe = warp_sum_u64(st_probe);
  status = __reduce_min_sync(kFull, status);
  if (lane == 0) {
    if (status != 0) atomicMin(const_cast<int32_t*>(cx.status), status);
    if (a.stats) atomicAdd(reinterpret_cast<unsigned long long*>(a.stats) + (size_t)p * 4, st_probe);
  }
}

// Commit warp `which` of kCommitWarps: the LRU commits of the requests routed to replicas
// i % kCommitWarps == which, in request order.  Commits on different replicas touch different
// bits of the mask words (set and cleared by reductions) and different recency lists, so the
// warps need no order among themselves; `progress[which]` says how far this one has got, and a
// request counts as committed once every warp has passed it.
template <typename MaskT>
__device__ __forceinline__ void commit_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p,
                                            uint32_t lane, uint32_t which) {
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R;
  const uint32_t N = a.tr.n_req;
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  MaskT* mask = cx.mask;
  uint32_t* lru_next = cx.lru_next;
  const uint8_t* route_log = cx.route_log;
  int32_t status = 0;
  unsigned long long st_evict = 0;
  const unsigned long long evict_guard_max = (unsigned long long)N + a.tr.n_ids / 16u + 64u;
  const uint32_t end = a.first + a.count;
  uint32_t jobs_seen = a.first;
  // a victim's block occurs again in request q soon after r: tell the gate warp
  auto mark_hit = [&](uint32_t q) { cx.evhit[q % kHitRing] = q; };

  PROF_BEGIN();
  for (uint32_t r = a.first; r < end; ++r) {
    if ((int32_t)(jobs_seen - (r + 1)) < 0) {
      jobs_seen = wait_counter(sm.jobs, r + 1, sm.abort_flag, a.poll_limit, status);
      if ((int32_t)(jobs_seen - (r + 1)) < 0) break;        // gave up
    }
    smem_order();
    PROF_LAP(0);
    const uint2 job2 = sm.job[r % kJobRing];
    const uint32_t job = job2.x;
    const uint32_t istar = job & 0xFFu;
    if (istar % kCommitWarps != which) {                    // another warp's replica
      if (lane == 0) sm.progress[which] = r + 1;
      PROF_LAP(4);
      continue;
    }
    const uint32_t slot = (job >> 8) & 0xFFu, n = job >> 16;
    const MaskT bit = (MaskT)(((MaskT)1) << istar);
    const uint32_t* sid = cx.st_ids + slot * kStageBlocks;
    const MaskT* smk = cx.st_mk + slot * kStageBlocks;

    // ---- how many blocks the commit inserts (the probe counted the blocks already present on
    //      the replica) and how many it has to evict first
    const uint32_t missing = n - (cx.st_hits[slot * R + istar] >> 16);
    uint32_t occ = sm.occ[istar] + missing;
    uint32_t need = occ > a.m.C ? (uint32_t)(occ - a.m.C) : 0u;
    PROF_ADD(12, need > 0 ? 1 : 0);
    PROF_ADD(15, need);
    uint32_t evicted = 0;
    if (need > 0) {
      uint32_t cr = sm.curreq[istar];
      int32_t cp = sm.curpos[istar];
      bool clean = false;
      // clean case: the scout's ring already holds `need` entries, none of them void or touched
      // again since it was listed; then exactly these are the victims
      if (sm.act[istar] && need <= 96u) {
        const uint32_t head = sm.ring_head[istar];
        if (sm.ring_tail[istar] - head >= need) {
          smem_order();
          const uint4* lst = sm.lst + (size_t)istar * kListCap;
          uint4 v0 = make_uint4(0, kNone, 0, 0), v1 = v0, v2 = v0;
          bool odd = false;
          auto look = [&](uint32_t idx, uint4& v) {
            if (idx < need) {
              const uint32_t e = (head + idx) & (kListCap - 1);
              v = a.lists_in_smem ? lst[e] : __ldcg(lst + e);
              odd = odd || v.y <= r || v.w < cr || (v.w == cr && (int32_t)v.z > cp);
            }
          };
          look(lane, v0);
          if (need > 32u) look(lane + 32u, v1);
          if (need > 64u) look(lane + 64u, v2);
          if (!__any_sync(kFull, odd)) {
            if (lane < need) { mask_clear_bit<MaskT>(mask, v0.x, bit); if (v0.y - (r + 1) < kWindow) mark_hit(v0.y); }
            if (lane + 32u < need) { mask_clear_bit<MaskT>(mask, v1.x, bit); if (v1.y - (r + 1) < kWindow) mark_hit(v1.y); }
            if (lane + 64u < need) { mask_clear_bit<MaskT>(mask, v2.x, bit); if (v2.y - (r + 1) < kWindow) mark_hit(v2.y); }
            // the eviction cursor moves behind the last victim
            const uint32_t li = need - 1;
            if (lane == (li & 31u)) {
              const uint4 le = li < 32u ? v0 : li < 64u ? v1 : v2;
              sm.curreq[istar] = le.w;
              sm.curpos[istar] = (int32_t)le.z - 1;
            }
            if (lane == 0) sm.ring_head[istar] = head + need;
            evicted = need;
            need = 0;
            clean = true;
            PROF_ADD(8, 1);
          } else PROF_ADD(9, 1);
        } else PROF_ADD(10, 1);
      } else PROF_ADD(11, 1);
      if (!clean) {
        // victims from the ring the scout warp keeps for this replica, entry by entry
        if (sm.act[istar]) {
          const uint4* lst = sm.lst + (size_t)istar * kListCap;
          uint32_t head = sm.ring_head[istar];
          uint32_t last_e = kNone;   // ring slot of the last entry passed that was not void
          #pragma unroll 1
          while (need > 0) {
            uint32_t avail = sm.ring_tail[istar] - head;
            for (uint32_t polls = 0; avail == 0 && polls < a.ring_polls; ++polls) {
              __nanosleep(20);
              avail = sm.ring_tail[istar] - head;
              PROF_ADD(14, 1);
            }
            if (avail == 0) break;                          // the scout is behind: walk ourselves
            smem_order();
            const uint32_t m = min(avail, 32u);
            uint4 ent = make_uint4(0, kNone, 0, 0);
            bool live = false, unsure = false;
            if (lane < m) {
              const uint32_t e = (head + lane) & (kListCap - 1);
              ent = a.lists_in_smem ? lst[e] : __ldcg(lst + e);
              // entries the eviction cursor has already passed (after a walk of our own) are void
              live = !(ent.w < cr || (ent.w == cr && (int32_t)ent.z > cp));
              if (live && ent.y <= r) {
                if (ent.y == r) live = false;               // the block is in this very request
                else {                                      // it came back in between: look again
                  live = !touch_is_stale(a.tr, route_log, req[ent.w].off + ent.z, istar, r, istar);
                  unsure = true;                            // where it occurs next is not known here
                }
              }
            }
            const unsigned lv = __ballot_sync(kFull, live);
            const uint32_t cnt = __popc(lv);
            const bool mine = live && (uint32_t)__popc(lv & ((1u << lane) - 1u)) < need;
            if (mine) {
              mask_clear_bit<MaskT>(mask, ent.x, bit);
              if (unsure) { for (uint32_t q = r + 1; q <= r + kWindow; ++q) mark_hit(q); }
              else if (ent.y - (r + 1) < kWindow) mark_hit(ent.y);
            }
            // entries passed: the whole round, or up to the last victim taken
            uint32_t passed = m, tk = cnt;
            if (cnt > need) {
              const unsigned take = __ballot_sync(kFull, mine);
              passed = 32u - (uint32_t)__clz((int)take);
              tk = need;
            }
            need -= tk;
            evicted += tk;
            // the cursor moves behind the last live entry passed (void ones lie behind it already)
            const unsigned seen = lv & (passed >= 32u ? kFull : ((1u << passed) - 1u));
            if (seen) last_e = (head + 31u - (uint32_t)__clz((int)seen)) & (kListCap - 1);
            head += passed;
          }
          if (last_e != kNone) {
            const uint4 le = a.lists_in_smem ? lst[last_e] : __ldcg(lst + last_e);
            cr = le.w;
            cp = (int32_t)le.z - 1;
          }
          if (lane == 0) sm.ring_head[istar] = head;
        }
        PROF_ADD(13, need > 0 ? 1 : 0);
        // whatever is still needed: walk the recency order from the cursor and validate touches here
        uint32_t coff = (cr != kNone && need > 0) ? req[cr].off : 0u;
        unsigned long long guard = 0;
        #pragma unroll 1
        while (need > 0) {
          if (++guard > evict_guard_max) { status = -6; break; }
          if (cp < 0) {  // this request is used up: go to the next one routed here
            const uint32_t nx = (cr == kNone) ? kNone : lru_next[cr];
            if (nx == kNone) { status = -6; break; }
            cr = nx;
            const ReqRec cre = req[cr];
            coff = cre.off;
            cp = (int32_t)cre.nblk - 1;
            continue;
          }
          // examine 32 touches, deepest position first
          const int32_t k = cp - (int32_t)lane;
          bool live = false;
          uint32_t vid = 0, nxr = kNone;
          if (k >= 0) {
            const uint32_t g = coff + (uint32_t)k;
            vid = ids[g];
            uint2 c = a.tr.occ_next[g];
            live = true;
            #pragma unroll 1
            while (c.x != kNone && c.y <= r) {       // later occurrences of the block, up to r
              const uint32_t rr = (c.y == r) ? istar : (uint32_t)route_log[c.y];
              if (rr == istar) { live = false; break; }
              c = a.tr.occ_next[c.x];
            }
            if (live && c.x != kNone) nxr = c.y;     // its next occurrence after r
          }
          const unsigned lv = __ballot_sync(kFull, live);
          const uint32_t cnt = __popc(lv);
          // the first `need` live touches in lane order are the victims
          const bool mine = live && (uint32_t)__popc(lv & ((1u << lane) - 1u)) < need;
          const unsigned take = __ballot_sync(kFull, mine);
          if (mine) {
            mask_clear_bit<MaskT>(mask, vid, bit);
            if (nxr - (r + 1) < kWindow) mark_hit(nxr);
          }
          cp -= (cnt <= need) ? 32 : 32 - __clz((int)take);
          const uint32_t tk = __popc(take);
          need -= tk;
          evicted += tk;
        }
        if (lane == 0) { sm.curreq[istar] = cr; sm.curpos[istar] = cp; }
      }
    }
    occ -= evicted;
    st_evict += evicted;
    PROF_LAP(1);

    // ---- set the replica's bit on the blocks the request inserts
    #pragma unroll 1
    for (uint32_t c = 0; c < n; c += 32) {
      const uint32_t k = c + lane;
      if (k < n) {
        uint32_t id;
        MaskT mv;
        if (c < kStageBlocks) { id = sid[k]; mv = smk[k]; }
        else { id = ids[job2.y + k]; mv = 0; }     // beyond the stage: set the bit without looking
        if (!(mv & bit)) mask_set_bit<MaskT>(mask, id, bit);
      }
    }
    __syncwarp();
    PROF_LAP(2);

    if (lane == 0) {
      sm.occ[istar] = occ;
      // recency order of the replica: append this request
      const uint32_t lt = sm.lrutail[istar];
      if (lt != kNone) lru_next[lt] = r;
      lru_next[r] = kNone;
      if (sm.curreq[istar] == kNone) { sm.curreq[istar] = r; sm.curpos[istar] = (int32_t)n - 1; }
      sm.lrutail[istar] = r;
      // hand the replica to the scout warp once its cache is close to full (before that no
      // eviction has happened here, so the scout starts from the eviction cursor)
      if (!sm.act[istar] && (uint64_t)occ + kPostMargin >= a.m.C) {
        sm.scan_cr[istar] = sm.curreq[istar];
        sm.scan_cp[istar] = sm.curpos[istar];
        __threadfence_block();
        sm.act[istar] = 1;
      }
      __threadfence_block();
      sm.progress[which] = r + 1;                         // request r is committed
    }
    __syncwarp();
    PROF_LAP(3);
  }
  PROF_END(48);
  status = __reduce_min_sync(kFull, status);
  if (lane == 0) {
    if (status != 0) atomicMin(const_cast<int32_t*>(cx.status), status);
    if (a.stats) atomicAdd(reinterpret_cast<unsigned long long*>(a.stats) + (size_t)p * 4 + 3, st_evict);
  }
}

// Roles of the twelve warps of a candidate.  Warp w issues from scheduler w % 4 of the SM, and a
// scheduler's instruction cache is small, so warps that run the same code sit on one scheduler:
//   scheduler 0: route, expiry, scout     scheduler 1: gate, service, scout
//   scheduler 2: probe, probe             scheduler 3: commit, commit, commit
enum Role : uint32_t { kRoleRoute, kRoleGate, kRoleProbe, kRoleScout, kRoleService, kRoleExpiry, kRoleCommit, kRoleNone };
constexpr uint32_t kReplayWarps = 12;
constexpr uint32_t kReplayThreads = 32 * kReplayWarps;
__device__ __forceinline__ void role_of(uint32_t warp, Role& role, uint32_t& which) {
  const uint32_t sched = warp & 3u, k = warp >> 2;
  which = k;
  if (sched == 0) role = k == 0 ? kRoleRoute : k == 1 ? kRoleExpiry : kRoleScout;
  else if (sched == 1) { role = k == 0 ? kRoleGate : k == 1 ? kRoleService : kRoleScout; which = 0; }
  else if (sched == 2) { role = k < kProbes ? kRoleProbe : (kServices == 2 && k == 2 ? kRoleService : kRoleNone); if (role == kRoleService) which = 1; }
  else role = k < kCommitWarps ? kRoleCommit : kRoleNone;
  if (role == kRoleScout) which = sched == 0 ? 0 : 1;      // scout 0 and scout 1
}
static_assert(kScouts == 2 && kProbes <= 3 && kCommitWarps <= 3 && kServices <= 2, "role map");
constexpr int kReplayMinCtas = 2;   // registers capped so that two candidates share an SM

template <typename MaskT, bool kBaseline>
__global__ void __launch_bounds__(kReplayThreads, kReplayMinCtas) replay_kernel(const ReplayArgs a) {
  const uint32_t p = blockIdx.x;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t R = a.m.R, S = a.m.S, K = a.m.K, G = a.m.G;
  const uint32_t N = a.tr.n_req;
  const uint32_t RS = R * S;

  unsigned char* st = a.states + (size_t)p * a.lay.bytes;
  CandHeader* hdr = reinterpret_cast<CandHeader*>(st);
  RepState* g_rep = reinterpret_cast<RepState*>(st + a.lay.rep_off);
  double* g_slot = reinterpret_cast<double*>(st + a.lay.slot_off);     // [R*S] slot free times

  extern __shared__ __align__(16) unsigned char smem_raw[];
  Ctx<MaskT> cx;
  Smem& sm = cx.sm;
  sm.rtt = reinterpret_cast<double*>(smem_raw);            // [G*R]
  sm.wrtt = sm.rtt + (size_t)G * R;                        // [G*R]  w_net * rtt
  sm.w = sm.wrtt + (size_t)G * R;                          // [K]
  sm.load = reinterpret_cast<long long*>(sm.w + K);        // [R]
  sm.cnt = sm.load + R;                                    // [R]
  sm.exp_sum = sm.cnt + R;                                 // [kExpRing][R]
  double* dnext = reinterpret_cast<double*>(sm.exp_sum + (size_t)kExpRing * R);
  // slot free times (in shared memory when they fit, else they stay in global memory)
  cx.free_at = g_slot;
  if (a.slots_in_smem) { cx.free_at = dnext; dnext += RS; }
  sm.occ = reinterpret_cast<uint32_t*>(dnext);             // [R]
  sm.curreq = sm.occ + R;
  sm.curpos = reinterpret_cast<int32_t*>(sm.curreq + R);
  sm.lrutail = reinterpret_cast<uint32_t*>(sm.curpos + R);
  uint32_t* unext = sm.lrutail + R;
  sm.progress = unext;                                     // [kCommitWarps] (<= 3)
  cx.route = unext + 3;
  cx.status = reinterpret_cast<volatile int32_t*>(unext + 4);
  cx.hit_slot = unext + 5;
  sm.routed = unext + 6;
  sm.exp_ready = unext + 7;
  sm.abort_flag = unext + 8;
  sm.jobs = unext + 9;
  sm.serviced = unext + 10;                                // [kServices] (<= 2)
  sm.route_ring = unext + 12;                              // [kRouteRing]
  sm.job = reinterpret_cast<uint2*>(sm.route_ring + kRouteRing);   // [kJobRing] (8-byte aligned: 4R + 12 + kRouteRing words after an aligned start)
  cx.evhit = reinterpret_cast<uint32_t*>(sm.job + kJobRing);       // [kHitRing]
  sm.act = const_cast<uint32_t*>(cx.evhit) + kHitRing;
  sm.ring_head = sm.act + R;
  sm.ring_tail = sm.ring_head + R;
  sm.scan_cr = sm.ring_tail + R;
  sm.scan_cp = reinterpret_cast<volatile int32_t*>(sm.scan_cr + R);
  {
    uint32_t* after = const_cast<uint32_t*>(sm.scan_cr) + 2 * (size_t)R;
    cx.st_ready = after;
    cx.probe_gone = after + kStageDepth;
    cx.st_hits = after + kStageDepth + 1;
    cx.st_ids = cx.st_hits + (kStageDepth + 2) * (size_t)R;
    after = cx.st_ids + (kStageDepth + 2) * (size_t)kStageBlocks;
    const uintptr_t a8 = (reinterpret_cast<uintptr_t>(after) + 7) & ~(uintptr_t)7;
    cx.st_ab = reinterpret_cast<double*>(a8);
    cx.st_where = reinterpret_cast<unsigned long long*>(cx.st_ab + (kStageDepth + 2) * (size_t)R);
    {
      const uintptr_t m16 = (reinterpret_cast<uintptr_t>(cx.st_where + (kStageDepth + 2)) + 15) & ~(uintptr_t)15;
      cx.st_meta = reinterpret_cast<uint4*>(m16);
    }
    cx.st_mk = reinterpret_cast<MaskT*>(cx.st_meta + (kStageDepth + 2));
    after = reinterpret_cast<uint32_t*>(cx.st_mk + (kStageDepth + 2) * (size_t)kStageBlocks);
    const uintptr_t al = (reinterpret_cast<uintptr_t>(after) + 15) & ~(uintptr_t)15;
    sm.lst = a.lists_in_smem ? reinterpret_cast<uint4*>(al)
                             : a.evict_lists + (size_t)p * R * kListCap;
  }
  cx.mask = reinterpret_cast<MaskT*>(a.masks + (size_t)p * a.mask_stride);
  cx.slot_kv = reinterpret_cast<unsigned long long*>(st + a.lay.slot_kv_off);
  cx.hdr = hdr;
  cx.finish_log = a.finish_log ? a.finish_log + (size_t)p * N : nullptr;
  cx.exp_head = a.exp_head + (size_t)p * N;
  cx.exp_rec = a.exp_rec + (size_t)p * N;
  cx.lru_next = a.lru_next + (size_t)p * N;
  cx.route_log = a.route_log + (size_t)p * a.route_log_stride;

  if (a.check_order && hdr->processed != a.first) {   // uniform over the CTA
    if (threadIdx.x == 0) {
      hdr->status = -8;
      if (a.status_out) a.status_out[p] = -8;
    }
    return;
  }

  for (uint32_t i = threadIdx.x; i < G * R; i += blockDim.x) {
    const double v = a.rtt[i];
    sm.rtt[i] = v;
    sm.wrtt[i] = __dmul_rn(a.params[(size_t)p * K], v);   // first product of the score
  }
  for (uint32_t i = threadIdx.x; i < K; i += blockDim.x) sm.w[i] = a.params[(size_t)p * K + i];
  for (uint32_t i = threadIdx.x; i < R; i += blockDim.x) {
    const RepState rs = g_rep[i];
    sm.load[i] = rs.load; sm.cnt[i] = rs.cnt; sm.occ[i] = rs.occ;
    sm.curreq[i] = rs.cur_req; sm.curpos[i] = rs.cur_pos; sm.lrutail[i] = rs.lru_tail;
    sm.act[i] = 0; sm.ring_head[i] = 0; sm.ring_tail[i] = 0;
  }
  if (a.slots_in_smem)
    for (uint32_t x = threadIdx.x; x < RS; x += blockDim.x) cx.free_at[x] = g_slot[x];
  if (threadIdx.x == 0) {
    *cx.status = 0; *cx.probe_gone = 0; *sm.abort_flag = 0;
    *sm.routed = a.first; *sm.exp_ready = a.first; *sm.jobs = a.first;
    sm.serviced[0] = a.first; if (kServices > 1) sm.serviced[1] = a.first;
  }
  if (cx.finish_log && threadIdx.x == 32) {
    // the trace may have grown since the last batch: requests that were to complete after its
    // old end are filed under the first request, not yet replayed, that arrives at or after
    // their finish time; the rest stay chained
    const double scale = a.scales ? a.scales[p] : a.scale;
    const double t_last = __dmul_rn(scale, a.tr.ts[N - 1]);
    uint32_t e = hdr->overflow - 1u, keep = kNone;
    #pragma unroll 1
    for (uint32_t guard = 0; e != kNone && guard < N; ++guard) {
      uint4 rec = cx.exp_rec[e];
      const uint32_t nxt = rec.x;
      const double f = cx.finish_log[e];
      if (e + 1 < N && t_last >= f) {
        const uint32_t x = first_arrival_at_or_after(a.tr.ts, scale, f, max(e + 1u, a.first), N - 1);
        rec.x = cx.exp_head[x];
        cx.exp_head[x] = e;
      } else {
        rec.x = keep;
        keep = e;
      }
      cx.exp_rec[e] = rec;
      e = nxt;
    }
    hdr->overflow = keep + 1u;
  }
  if (threadIdx.x < kCommitWarps) sm.progress[threadIdx.x] = a.first;
  if (threadIdx.x < kStageDepth) cx.st_ready[threadIdx.x] = 0;
  if (threadIdx.x < kJobRing) sm.job[threadIdx.x] = make_uint2(0u, 0u);
  if (threadIdx.x < kHitRing) cx.evhit[threadIdx.x] = kNone;
  __syncthreads();

  Role role;
  uint32_t which;
  role_of(warp, role, which);
  if (role == kRoleRoute) route_warp<MaskT, kBaseline>(a, cx, p, lane);
  else if (role == kRoleGate) gate_warp<MaskT, kBaseline>(a, cx, p, lane);
  else if (role == kRoleCommit) commit_warp<MaskT>(a, cx, p, lane, which);
  else if (role == kRoleProbe) probe_warp<MaskT, kBaseline>(a, cx, p, lane, which);
  else if (role == kRoleService) service_warp<MaskT, kBaseline>(a, cx, p, lane, which);
  else if (role == kRoleExpiry)
    expiry_warp<kBaseline>(a, sm, cx.exp_head, cx.exp_rec, sm.abort_flag, cx.status, p, lane);
  else if (role == kRoleScout) scout_warp<MaskT>(a, sm, cx.lru_next, cx.route_log, lane, which);
  __syncthreads();

  // ---- write the small state back
  for (uint32_t i = threadIdx.x; i < R; i += blockDim.x) {
    RepState rs;
    rs.load = sm.load[i]; rs.cnt = sm.cnt[i]; rs.occ = sm.occ[i];
    rs.cur_req = sm.curreq[i]; rs.cur_pos = sm.curpos[i]; rs.lru_tail = sm.lrutail[i];
    g_rep[i] = rs;
  }
  if (a.slots_in_smem)
    for (uint32_t x = threadIdx.x; x < RS; x += blockDim.x) g_slot[x] = cx.free_at[x];
  if (threadIdx.x == 0) {
    const int32_t status = *cx.status;
    hdr->processed = a.first + a.count;
    if (status != 0) hdr->status = status;
    if (a.status_out && (status != 0 || !a.check_order)) a.status_out[p] = status;
  }
}

// ------------------------------------------------------------------------------- reset
// One warp per appended request: a block whose previous occurrence belongs to an earlier batch
// becomes that occurrence's successor.
__global__ void link_occurrences_kernel(TraceView tr, uint32_t first_new, uint32_t n_new,
                                        uint32_t ids_before, uint2* occ_next) {
  const uint32_t k = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  if (k >= n_new) return;
  const uint32_t r = first_new + k;
  const ReqRec q = tr.req[r];
  for (uint32_t c = threadIdx.x % 32; c < q.nblk; c += 32) {
    const uint2 pv = tr.occ_prev[q.off + c];
    if (pv.x != kNone && pv.x < ids_before) occ_next[pv.x] = make_uint2(q.off + c, r);
  }
}

__global__ void reset_states_kernel(unsigned char* states, StateLayout lay, uint32_t R, uint32_t S,
                                    uint32_t n_cand) {
  const uint32_t p = blockIdx.x;
  if (p >= n_cand) return;
  unsigned char* st = states + (size_t)p * lay.bytes;
  if (threadIdx.x == 0) {
    CandHeader h = {};
    *reinterpret_cast<CandHeader*>(st) = h;
  }
  RepState* rep = reinterpret_cast<RepState*>(st + lay.rep_off);
  for (uint32_t i = threadIdx.x; i < R; i += blockDim.x) {
    RepState rs;
    rs.load = 0; rs.cnt = 0; rs.occ = 0; rs.cur_req = kNone; rs.cur_pos = -1;
    rs.lru_tail = kNone;
    rep[i] = rs;
  }
  double* slot = reinterpret_cast<double*>(st + lay.slot_off);
  const uint32_t RS = R * S;
  unsigned long long* kv = reinterpret_cast<unsigned long long*>(st + lay.slot_kv_off);
  for (uint32_t x = threadIdx.x; x < RS; x += blockDim.x) { slot[x] = 0.0; kv[x] = 0; }   // free from time 0
}

// ------------------------------------------------------------------------------ select
// Exact k-th smallest (k = ceil(0.95 n), nearest rank) of n doubles by most-significant-digit
// radix selection on order-preserving 64-bit keys; one CTA per (candidate, metric).
__device__ __forceinline__ uint64_t key_of(double v) {
  const uint64_t b = (uint64_t)__double_as_longlong(v);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ULL);
}
__device__ __forceinline__ double value_of(uint64_t k) {
  const uint64_t b = (k >> 63) ? (k & 0x7FFFFFFFFFFFFFFFULL) : ~k;
  return __longlong_as_double((long long)b);
}

constexpr int kSelectThreads = 1024;

__global__ void __launch_bounds__(kSelectThreads) select_p95_kernel(const SelectArgs a) {
  const uint32_t p = blockIdx.x;
  const double* v = (blockIdx.y == 0 ? a.ttft : a.e2e) + (size_t)p * a.stride;
  double* out = (blockIdx.y == 0 ? a.p95_ttft : a.p95_e2e) + p;
  const uint32_t n = a.n;
  __shared__ uint32_t hist[256];
  __shared__ uint64_t s_prefix;
  __shared__ uint32_t s_rank;
  if (n == 0) { if (threadIdx.x == 0) *out = 0.0; return; }
  if (threadIdx.x == 0) {
    s_prefix = 0;
    s_rank = (uint32_t)((95ull * n + 99ull) / 100ull) - 1u;  // 0-based rank
  }
  uint64_t have = 0;  // mask of the key bits fixed so far
  for (int shift = 56; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const uint64_t prefix = s_prefix;
    for (uint32_t base = threadIdx.x & ~31u; base < n; base += blockDim.x) {
      const uint32_t i = base + (threadIdx.x & 31u);
      const uint64_t k = (i < n) ? key_of(v[i]) : 0;
      const bool in = (i < n) && (k & have) == prefix;
      const uint32_t d = (uint32_t)(k >> shift) & 255u;
      // one atomic per distinct digit among the matching lanes of the warp
      const unsigned act = __ballot_sync(kFull, in);
      if (in) {
        const unsigned peers = __match_any_sync(act, d);
        if ((uint32_t)(__ffs((int)peers) - 1) == (threadIdx.x & 31u)) atomicAdd(&hist[d], __popc(peers));
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t rank = s_rank, d = 0;
      while (d < 255 && rank >= hist[d]) { rank -= hist[d]; ++d; }
      s_rank = rank;
      s_prefix = prefix | ((uint64_t)d << shift);
    }
    have |= (uint64_t)255 << shift;
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = value_of(s_prefix);
}

// ------------------------------------------------------------------------ baseline routes
// Per-request routes of the baselines that do not look at the simulator's state (paper Section
// 4): session affinity (the paper hashes the first 256 tokens of the prompt; the id of the first
// block stands for them: finaliser of the caller's 64-bit id, modulo R; replica 0 for a prompt
// without blocks) and random (one caller-supplied draw per request, modulo R).
__global__ void policy_routes_kernel(TraceView tr, uint32_t R, uint32_t affinity,
                                     const uint32_t* draws, uint8_t* route) {
  const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= tr.n_req) return;
  uint32_t i = 0;
  if (affinity) {
    const ReqRec q = tr.req[r];
    if (q.nblk > 0) i = (uint32_t)(mix64(tr.raw_id[tr.ids[q.off]]) % R);
  } else {
    i = draws[r] % R;
  }
  route[r] = (uint8_t)i;
}

// ------------------------------------------------------------------------ window objective
// Rolling-window objective of the tuning loop (paper Section 4: p95 TTFT of a rolling 128-request
// window with hop 32): window j covers requests [j*hop, j*hop + window); its value is the k-th
// smallest of them, k = ceil(0.95 window) (nearest rank).  One warp per window: the window's
// order-preserving keys are copied to the warp's piece of shared memory, padded to a power of two
// with the largest key, sorted by a bitonic network (exact for any input) and read at rank k-1.
constexpr int kWindowThreads = 128;                   // four windows in flight per CTA
constexpr uint32_t kWindowMax = 2048;                 // longest window (its keys: 16 KB per warp)

__global__ void __launch_bounds__(kWindowThreads) window_p95_kernel(const WindowArgs a,
                                                                    uint32_t wpad) {
  extern __shared__ __align__(16) unsigned char window_smem[];
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t warps = kWindowThreads / 32;
  uint64_t* keys = reinterpret_cast<uint64_t*>(window_smem) + (size_t)warp * wpad;
  const uint32_t p = blockIdx.x;
  const double* v = a.values + (size_t)p * a.stride;
  double* out = a.win_p95 + (size_t)p * a.win_stride;
  const uint32_t W = a.window;
  const uint32_t rank = (uint32_t)((95ull * W + 99ull) / 100ull) - 1u;   // 0-based
  for (uint32_t j = blockIdx.y * warps + warp; j < a.n_win; j += gridDim.y * warps) {
    const double* wv = v + (size_t)j * a.hop;
    for (uint32_t i = lane; i < wpad; i += 32) keys[i] = i < W ? key_of(wv[i]) : ~0ull;
    __syncwarp();
    for (uint32_t size = 2; size <= wpad; size <<= 1) {
      for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
        for (uint32_t t = lane; t < wpad / 2; t += 32) {
          const uint32_t i = 2 * t - (t & (stride - 1));     // lower element of the t-th pair
          const bool ascending = (i & size) == 0;
          const uint64_t x = keys[i], y = keys[i + stride];
          if ((x > y) == ascending) { keys[i] = y; keys[i + stride] = x; }
        }
        __syncwarp();
      }
    }
    if (lane == 0) out[j] = value_of(keys[rank]);
    __syncwarp();
  }
}

// The same for windows of up to 256 values, without shared memory and without sorting: only the
// largest W - k + 1 values matter for the k-th smallest (about 5 % of the window).  Every lane
// holds its NR keys (values lane, lane+32, ...) in registers, sorted descending; the warp then
// takes the maximum over the lanes' current tops W - k + 1 times (two reductions on the halves of
// the 64-bit keys), each time popping it from the lowest lane that holds it.
template <int NR>
__global__ void __launch_bounds__(kWindowThreads) window_p95_select_kernel(const WindowArgs a) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t warps = kWindowThreads / 32;
  const uint32_t p = blockIdx.x;
  const double* v = a.values + (size_t)p * a.stride;
  double* out = a.win_p95 + (size_t)p * a.win_stride;
  const uint32_t W = a.window;
  const uint32_t takes = W - (uint32_t)((95ull * W + 99ull) / 100ull) + 1u;   // the answer is the takes-th largest
  for (uint32_t j = blockIdx.y * warps + warp; j < a.n_win; j += gridDim.y * warps) {
    const double* wv = v + (size_t)j * a.hop;
    uint64_t k[NR];
#pragma unroll
    for (int i = 0; i < NR; ++i) {
      const uint32_t idx = lane + 32u * i;
      k[i] = idx < W ? key_of(wv[idx]) : 0ull;          // (0 is below the key of every double)
    }
    // sort the lane's keys descending (odd-even transposition over NR registers)
#pragma unroll
    for (int round = 0; round < NR; ++round) {
#pragma unroll
      for (int i = round & 1; i + 1 < NR; i += 2) {
        const uint64_t hi = k[i] > k[i + 1] ? k[i] : k[i + 1];
        const uint64_t lo = k[i] > k[i + 1] ? k[i + 1] : k[i];
        k[i] = hi; k[i + 1] = lo;
      }
    }
    uint64_t best = 0;
    for (uint32_t t = 0; t < takes; ++t) {
      const uint32_t hi = (uint32_t)(k[0] >> 32), lo = (uint32_t)k[0];
      const uint32_t mh = __reduce_max_sync(kFull, hi);
      const uint32_t ml = __reduce_max_sync(kFull, hi == mh ? lo : 0u);
      best = ((uint64_t)mh << 32) | ml;
      const unsigned owners = __ballot_sync(kFull, k[0] == best);
      if (lane == (uint32_t)__ffs((int)owners) - 1u) {   // pop it from one lane
#pragma unroll
        for (int i = 0; i + 1 < NR; ++i) k[i] = k[i + 1];
        k[NR - 1] = 0ull;
      }
    }
    if (lane == 0) out[j] = value_of(best);
  }
}

// Smallest window value of every candidate and the first window that attains it.
__global__ void __launch_bounds__(256) window_best_kernel(const WindowArgs a) {
  const uint32_t p = blockIdx.x;
  const double* w = a.win_p95 + (size_t)p * a.win_stride;
  __shared__ uint64_t s_key[256];
  __shared__ uint32_t s_idx[256];
  uint64_t bk = ~0ull;
  uint32_t bi = kNone;
  for (uint32_t j = threadIdx.x; j < a.n_win; j += blockDim.x) {
    const uint64_t k = key_of(w[j]);
    if (k < bk) { bk = k; bi = j; }            // ascending j per thread: first minimum kept
  }
  s_key[threadIdx.x] = bk; s_idx[threadIdx.x] = bi;
  __syncthreads();
  for (uint32_t d = 128; d > 0; d >>= 1) {
    if (threadIdx.x < d) {
      const uint64_t ok = s_key[threadIdx.x + d];
      const uint32_t oi = s_idx[threadIdx.x + d];
      if (ok < s_key[threadIdx.x] || (ok == s_key[threadIdx.x] && oi < s_idx[threadIdx.x])) {
        s_key[threadIdx.x] = ok; s_idx[threadIdx.x] = oi;
      }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    a.best[p] = a.n_win ? value_of(s_key[0]) : 0.0;
    if (a.best_win) a.best_win[p] = s_idx[0];
  }
}

// ------------------------------------------------------------------------------ digest
// Per replica: occupancy and the sum over cached blocks of mix64(id ^ mix64(seq*65536+pos)).
// A block's latest touch on its replica is cached iff it lies at or after the eviction cursor.
__global__ void __launch_bounds__(256) digest_kernel(const DigestArgs a) {
  const uint32_t p = blockIdx.x;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warp = (blockIdx.y * blockDim.x + threadIdx.x) >> 5;
  const uint32_t n_warps = (gridDim.y * blockDim.x) >> 5;
  const unsigned char* st = a.states + (size_t)p * a.lay.bytes;
  const CandHeader* hdr = reinterpret_cast<const CandHeader*>(st);
  const RepState* rep = reinterpret_cast<const RepState*>(st + a.lay.rep_off);
  const uint8_t* route_log = a.route_log + (size_t)p * a.route_log_stride;
  const uint32_t done = hdr->processed;
  if (done == 0) return;
  unsigned long long* dg = reinterpret_cast<unsigned long long*>(a.digest) + (size_t)p * a.m.R * 2;
  for (uint32_t n = warp; n < done; n += n_warps) {
    const uint32_t i = route_log[n];
    const uint32_t cr = rep[i].cur_req;
    const int32_t cp = rep[i].cur_pos;
    if (cr == kNone || n < cr) continue;
    const ReqRec rec = a.tr.req[n];
    unsigned long long sum = 0, cnt = 0;
    for (uint32_t k = lane; k < rec.nblk; k += 32) {
      if (n == cr && (int32_t)k > cp) continue;
      const uint32_t g = rec.off + k;
      if (touch_is_stale(a.tr, route_log, g, i, done - 1, route_log[done - 1])) continue;
      const uint64_t id = a.tr.raw_id[a.tr.ids[g]];
      sum += mix64(id ^ mix64((uint64_t)n * 65536ULL + k));
      cnt += 1;
    }
    sum = warp_sum_u64(sum);
    cnt = warp_sum_u64(cnt);
    if (lane == 0 && cnt) {
      atomicAdd(&dg[2 * i], cnt);
      atomicAdd(&dg[2 * i + 1], sum);
    }
  }
}

template <typename MaskT>
size_t replay_smem_bytes(ReplayArgs& a) {
  const size_t rs = (size_t)a.m.R * a.m.S;
  const size_t list_bytes = (size_t)a.m.R * kListCap * sizeof(uint4);
  a.slots_in_smem = rs * 8 <= 40 * 1024 ? 1u : 0u;
  a.lists_in_smem = list_bytes <= 64 * 1024 ? 1u : 0u;
  size_t smem = (2 * (size_t)a.m.G * a.m.R + a.m.K + (2 + kExpRing) * (size_t)a.m.R) * sizeof(double) +
                (9 * (size_t)a.m.R + 12 + kRouteRing + 2 * kJobRing + kHitRing) * sizeof(uint32_t) + 16 +
                (kStageDepth + 2) * (sizeof(unsigned long long) + sizeof(uint4)) + 16 +
                (kStageDepth + 1 + (kStageDepth + 2) * ((size_t)a.m.R + kStageBlocks)) * sizeof(uint32_t) +
                8 + (kStageDepth + 2) * (size_t)a.m.R * sizeof(double) +
                (kStageDepth + 2) * kStageBlocks * sizeof(MaskT) + 8;
  if (a.slots_in_smem) smem += rs * 8;
  if (a.lists_in_smem) smem += list_bytes;
  smem = (smem + 15) / 16 * 16;
  return smem;
}

template <typename MaskT, bool kBaseline>
cudaError_t launch_replay_tb(ReplayArgs a, uint32_t n_cand, cudaStream_t st) {
  const size_t smem = replay_smem_bytes<MaskT>(a);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(replay_kernel<MaskT, kBaseline>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  // several candidates share an SM (P is usually larger than the SM count): ask for the largest
  // shared-memory carve-out so that the per-CTA footprint, not the default split, decides
  {
    cudaError_t e = cudaFuncSetAttribute(replay_kernel<MaskT, kBaseline>,
                                         cudaFuncAttributePreferredSharedMemoryCarveout,
                                         (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
  }
  replay_kernel<MaskT, kBaseline><<<n_cand, kReplayThreads, smem, st>>>(a);
  return cudaGetLastError();
}

template <typename MaskT>
cudaError_t launch_replay_t(const ReplayArgs& a, uint32_t n_cand, cudaStream_t st) {
  if (a.queue_in_requests || a.forced_route || a.rep_prefill_ms || a.rep_tpot_ms ||
      a.decode_slowdown > 0.0 || a.kv_budget > 0 || a.rtt_ewma || a.proxy_index)
    return launch_replay_tb<MaskT, true>(a, n_cand, st);
  return launch_replay_tb<MaskT, false>(a, n_cand, st);
}

}  // namespace

template <typename MaskT>
int replay_occupancy_t(ReplayArgs a, size_t* smem_out) {
  const size_t smem = replay_smem_bytes<MaskT>(a);
  *smem_out = smem;
  cudaFuncSetAttribute(replay_kernel<MaskT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  cudaFuncSetAttribute(replay_kernel<MaskT, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                       (int)cudaSharedmemCarveoutMaxShared);
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, replay_kernel<MaskT, false>, (int)kReplayThreads,
                                                    smem) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return n;
}

int replay_occupancy(const Model& m, uint64_t* smem_bytes) {
  ReplayArgs a = {};
  a.m = m;
  int n;
  size_t smem = 0;
  switch (mask_bytes_for(m.R)) {
    case 1: n = replay_occupancy_t<uint8_t>(a, &smem); break;
    case 2: n = replay_occupancy_t<uint16_t>(a, &smem); break;
    case 4: n = replay_occupancy_t<uint32_t>(a, &smem); break;
    default: n = replay_occupancy_t<uint64_t>(a, &smem); break;
  }
  if (smem_bytes) *smem_bytes = smem;
  return n;
}

uint64_t evict_list_bytes(uint32_t n_replicas) {
  return (uint64_t)n_replicas * kListCap * sizeof(uint4);
}

uint32_t mask_bytes_for(uint32_t n_replicas) {
  return n_replicas <= 8 ? 1u : n_replicas <= 16 ? 2u : n_replicas <= 32 ? 4u : 8u;
}

cudaError_t launch_reset(unsigned char* masks, uint64_t mask_bytes_total, uint32_t* exp_head,
                         uint64_t exp_head_count, unsigned char* states, const StateLayout& lay,
                         const Model& m, uint32_t n_cand, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(masks, 0, mask_bytes_total, st);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(exp_head, 0xFF, exp_head_count * sizeof(uint32_t), st);   // kNone: empty lists
  if (e != cudaSuccess) return e;
  reset_states_kernel<<<n_cand, 128, 0, st>>>(states, lay, m.R, m.S, n_cand);
  return cudaGetLastError();
}

cudaError_t launch_link_occurrences(const TraceView& tr, uint32_t first_new, uint32_t n_new,
                                    uint32_t ids_before, uint2* occ_next, cudaStream_t st) {
  link_occurrences_kernel<<<(n_new + 7) / 8, 256, 0, st>>>(tr, first_new, n_new, ids_before, occ_next);
  return cudaGetLastError();
}

cudaError_t launch_replay(const ReplayArgs& a, uint32_t n_cand, cudaStream_t st) {
  switch (mask_bytes_for(a.m.R)) {
    case 1: return launch_replay_t<uint8_t>(a, n_cand, st);
    case 2: return launch_replay_t<uint16_t>(a, n_cand, st);
    case 4: return launch_replay_t<uint32_t>(a, n_cand, st);
    default: return launch_replay_t<uint64_t>(a, n_cand, st);
  }
}

cudaError_t launch_select(const SelectArgs& a, uint32_t n_cand, cudaStream_t st) {
  select_p95_kernel<<<dim3(n_cand, 2), kSelectThreads, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_policy_routes(const TraceView& tr, uint32_t R, bool affinity,
                                 const uint32_t* draws, uint8_t* route, cudaStream_t st) {
  policy_routes_kernel<<<(tr.n_req + 255) / 256, 256, 0, st>>>(tr, R, affinity ? 1u : 0u, draws, route);
  return cudaGetLastError();
}

#ifdef GORGO_PROF
cudaError_t prof_read(unsigned long long* out64, bool reset) {
  cudaError_t e = cudaMemcpyFromSymbol(out64, g_prof, sizeof(g_prof));
  if (e != cudaSuccess || !reset) return e;
  unsigned long long zero[64] = {};
  return cudaMemcpyToSymbol(g_prof, zero, sizeof(zero));
}
#endif

// ------------------------------------------------------------------ gather yardstick
// Every thread reads `per_thread` 32-byte sectors at pseudo-random positions of a buffer of
// `n_sectors` sectors (position = splitmix64 finaliser of a counter, so consecutive reads of one
// thread and the reads of neighbouring threads land on unrelated sectors) and keeps one word of
// each, eight reads in flight per thread.  What it measures is the rate at which this GPU serves
// independent 32-byte reads from a footprint of that size: DRAM sectors when the footprint is
// far larger than L2, L2 sectors when it fits.
__global__ void __launch_bounds__(256) gather_sectors_kernel(const uint4* buf, uint64_t n_sectors,
                                                             uint32_t per_thread, uint32_t* sink) {
  const uint64_t tid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint64_t n_threads = (uint64_t)gridDim.x * blockDim.x;
  uint32_t acc = 0;
  for (uint32_t it = 0; it < per_thread; it += 8) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const uint64_t c = ((uint64_t)(it + u) * n_threads + tid) * 0x9E3779B97F4A7C15ULL;
      const uint64_t sector = mix64(c) % n_sectors;
      v[u] = __ldcg(buf + sector * 2);                  // first half of the 32-byte sector
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) acc += v[u].x ^ v[u].w;
  }
  if (acc == 0x12345u) *sink = acc;                     // keeps the loads alive
}

cudaError_t launch_gather(const void* buf, uint64_t n_sectors, uint32_t per_thread, uint32_t blocks,
                          uint32_t* sink, cudaStream_t st) {
  gather_sectors_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint4*>(buf), n_sectors,
                                                per_thread, sink);
  return cudaGetLastError();
}

uint32_t window_max() { return kWindowMax; }

cudaError_t launch_window(const WindowArgs& a, uint32_t n_cand, cudaStream_t st) {
  if (a.n_win > 0) {
    uint32_t wpad = 1;
    while (wpad < a.window) wpad <<= 1;
    const uint32_t warps = kWindowThreads / 32;
    const size_t smem = (size_t)warps * wpad * sizeof(uint64_t);
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(window_p95_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    const uint32_t groups_needed = (a.n_win + warps - 1) / warps;
    const uint32_t groups = groups_needed < 1024u ? groups_needed : 1024u;
    const dim3 grid(n_cand, groups);
    if (wpad <= 32) window_p95_select_kernel<1><<<grid, kWindowThreads, 0, st>>>(a);
    else if (wpad == 64) window_p95_select_kernel<2><<<grid, kWindowThreads, 0, st>>>(a);
    else if (wpad == 128) window_p95_select_kernel<4><<<grid, kWindowThreads, 0, st>>>(a);
    else if (wpad == 256) window_p95_select_kernel<8><<<grid, kWindowThreads, 0, st>>>(a);
    else window_p95_kernel<<<grid, kWindowThreads, smem, st>>>(a, wpad);
  }
  window_best_kernel<<<n_cand, 256, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_digest(const DigestArgs& a, uint32_t n_cand, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(a.digest, 0, (size_t)n_cand * a.m.R * 2 * sizeof(uint64_t), st);
  if (e != cudaSuccess) return e;
  const uint32_t chunks = 64;
  digest_kernel<<<dim3(n_cand, chunks), 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace gorgo

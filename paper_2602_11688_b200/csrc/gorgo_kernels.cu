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
//  * in-flight accounting through per-slot FIFO chains (finish times on one slot never
//    decrease), with the earliest finish per replica cached so the common case is one compare.
// Requests are strictly ordered inside a candidate and every step depends on the one before, so
// a replay is bound by the latency of that chain, not by bandwidth.  One CTA of five warps
// replays one candidate and the warps split the chain:
//   decide  queue signal, score (Eq. 3), argmin, service model, outputs;
//   cache   validates the staged prefix hits, sizes and performs the eviction, recency list;
//   probe   runs up to three requests ahead: reads block ids and mask words, probes them and
//           stages hits and the hit-dependent part of the score in shared memory;
//   scout   (two warps) validate touches ahead of every replica's eviction cursor and keep a
//           ring of ready victims per replica.
// A staged read may predate the commits of the last three requests; the cache warp knows which
// of those commits can have touched the request (shared block, or evicted block that occurs in
// it) and then repeats the read itself, so results never depend on the timing of the warps.
#include "gorgo_internal.h"

namespace gorgo {

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;

// Optional cycle accounting of the replay warps (build with -DGORGO_PROF): every warp adds the
// clock cycles it spends between the marks GORGO_PT(i) to counter i of its role, lane 0 adds them
// to a global table at the end, `gorgo_prof_read` copies the table out.  Compiled out otherwise.
#ifdef GORGO_PROF
__device__ unsigned long long g_prof[256];
#define GORGO_PROF_DECL long long pf_t = clock64(); unsigned long long pf[16] = {0,0,0,0,0,0,0,0,0,0,0,0,0,0,0,0};
#define GORGO_PT(i) { const long long pf_n = clock64(); pf[i] += (unsigned long long)(pf_n - pf_t); pf_t = pf_n; }
#define GORGO_PC(i, v) { pf[i] += (v); }
#define GORGO_PROF_FLUSH(role) if (lane == 0) { for (int pf_i = 0; pf_i < 16; ++pf_i) atomicAdd(&g_prof[(role) * 16 + pf_i], pf[pf_i]); }
#else
#define GORGO_PROF_DECL
#define GORGO_PT(i)
#define GORGO_PC(i, v)
#define GORGO_PROF_FLUSH(role)
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
__device__ __forceinline__ double order_value(uint64_t k) {
  const uint64_t b = (k >> 63) ? (k & 0x7FFFFFFFFFFFFFFFULL) : ~k;
  return __longlong_as_double((long long)b);
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
// Mask words are read and written around L1: they are also changed by reductions in L2.
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
template <typename MaskT>
__device__ __forceinline__ void mask_store(MaskT* mask, uint32_t id, MaskT v) {
  __stcg(mask + id, v);
}
template <>
__device__ __forceinline__ void mask_store<uint8_t>(uint8_t* mask, uint32_t id, uint8_t v) {
  __stcg(reinterpret_cast<unsigned char*>(mask) + id, (unsigned char)v);
}
template <>
__device__ __forceinline__ void mask_store<uint16_t>(uint16_t* mask, uint32_t id, uint16_t v) {
  __stcg(reinterpret_cast<unsigned short*>(mask) + id, (unsigned short)v);
}
template <>
__device__ __forceinline__ void mask_store<uint64_t>(uint64_t* mask, uint32_t id, uint64_t v) {
  __stcg(reinterpret_cast<unsigned long long*>(mask) + id, (unsigned long long)v);
}

constexpr int kRegChunks = 8;                          // 32-block chunks of a request a probe warp holds
constexpr uint32_t kStageBlocks = kRegChunks * 32u;    // blocks of a request kept per stage
constexpr uint32_t kStageDepth = 8;                    // requests staged ahead of the cache warp
constexpr uint32_t kWindow = kStageDepth - 1;          // a staged read is at most this many commits old
constexpr uint32_t kStages = kStageDepth + 2;          // + two stages for the route warp's own probes
constexpr uint32_t kRouteRing = 32;                    // routed requests not yet served / committed
constexpr uint32_t kExpRing = 16;                      // requests whose expiries are staged ahead
constexpr uint32_t kInvalRing = 16;                    // > kWindow: requests whose staged read is void
constexpr uint32_t kApplyRing = 8;                     // commits checked but not yet applied
constexpr uint32_t kQueueWarps = 2;                    // replicas are split between them (i mod 2)
constexpr uint32_t kProbeWarps = 2;                    // requests are split between them (r mod 2)
constexpr uint32_t kScouts = 2;                        // scout warps (replicas split between them)
constexpr uint32_t kListCap = 256;                     // pre-validated eviction victims kept per replica
constexpr int kScoutBatches = 1;                       // touches examined per lane and scout round
constexpr uint32_t kPostMargin = 512;                  // start pre-validating when a cache is this close to full
constexpr uint32_t kSpinLimit = 1u << 24;              // polls after which a waiting warp gives up
constexpr uint32_t kPollNs = 20;                       // pause between polls: keeps the waiting warps
                                                       //   from flooding the shared-memory pipeline

// Words of the control block (shared memory) through which the warps of a candidate pace each
// other.  Counters hold request indices; they only grow.
constexpr uint32_t kCtlRouted = 0;      // requests < this have a route (route warp)
constexpr uint32_t kCtlApplied = 1;     // requests < this are fully committed to the cache state
constexpr uint32_t kCtlChecked = 2;     // requests < this have their eviction victims determined
constexpr uint32_t kCtlEnqueued = 3;    // requests < this have their commit handed to the apply warp
constexpr uint32_t kCtlAbort = 4;       // a warp ran into a limit: everybody stops
constexpr uint32_t kCtlStatus = 5;
constexpr uint32_t kCtlProbeGone = 6;   // probe warps that have stopped
constexpr uint32_t kCtlExp = 8;         // [kQueueWarps] requests < this have their expiries staged
constexpr uint32_t kCtlServed = kCtlExp + kQueueWarps;   // [kQueueWarps] requests < this are booked
constexpr uint32_t kCtlWords = (kCtlServed + kQueueWarps + 1u) & ~1u;

// Shared-memory view of one candidate's small state.
struct Smem {
  double* rtt; double* wrtt; double* w; double* minfin; long long* load;
  uint32_t* occ; uint32_t* curreq; int32_t* curpos;
  volatile uint32_t* lrutail;     // last request appended to a replica's recency list (apply warp)
  uint32_t* c_lrutail;            // last request routed to it as the check warp knows it
  uint32_t* chead;                // ring entries taken by the check warp (>= ring_head)
  volatile uint32_t* progress;    // the kCtlApplied word
  volatile uint32_t* abort;       // the kCtlAbort word
  // eviction rings, one per replica: filled by a scout warp, drained by the cache warp.
  // entry = (block id, request of the block's next occurrence after the entry was made or kNone,
  //          position of the touch in its request, request of the touch), in eviction order
  uint4* lst;                     // [R][kListCap]
  volatile uint32_t* act;         // cache -> scout: the replica's cache is close to full
  volatile uint32_t* ring_head;   // entries consumed and free for reuse (apply warp)
  volatile uint32_t* ring_tail;   // entries produced (scout warp)
  volatile uint32_t* scan_cr;     // scout's own cursor into the recency order (set at activation)
  volatile int32_t* scan_cp;
};

// Scout warp: for every replica whose cache is close to full it walks the recency order ahead
// of the eviction cursor and appends to the replica's ring the touches that are still the latest
// touch of their block (the coming eviction victims, in order).  The cache warp evicts from the
// ring instead of validating touches itself; entries that went stale after they were appended
// are recognised there by their next-occurrence field.
template <typename MaskT>
__device__ __forceinline__ void scout_warp(const ReplayArgs& a, const Smem& sm, const uint32_t* lru_next,
                           const uint8_t* route_log, uint32_t lane, uint32_t which) {
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  const uint32_t end = a.first + a.count;
  const uint32_t R = a.m.R;
  uint32_t idle = 0;
  uint32_t blocked0 = kNone - 1, blocked1 = kNone - 1;  // lru tail seen when the scan ran dry
  GORGO_PROF_DECL
  while (true) {
    const uint32_t prog = *sm.progress;
    if (prog >= end || *sm.abort) break;
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
      GORGO_PT(0)
      continue;
    }
    GORGO_PT(1)
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
      __threadfence_block();
      __syncwarp();
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
    GORGO_PT(2)
  }
  GORGO_PROF_FLUSH(11 + which)
}

// Everything the warps of one candidate share.
template <typename MaskT>
struct Ctx {
  Smem sm;
  MaskT* mask;
  uint4* qrec;
  uint32_t* lru_next;
  uint8_t* route_log;
  // per-slot state (shared or global memory)
  double *free_at, *q0_fin, *q1_fin;
  uint32_t *q0_tok, *q1_tok, *q2_idx, *tail, *qcnt;
  volatile uint32_t* ctl;         // [kCtlWords] control block
  volatile uint32_t* route_ring;  // [kRouteRing] replica | stage << 8 | prefix hit on it << 16
  long long* exp_sub;             // [kExpRing][R] tokens that stop being in flight at a request
  uint4* apply_ring;              // [kApplyRing][2] work items of the apply warp (ApplyItem)
  volatile uint32_t* inval;       // [kInvalRing] request (+1) that lost a cached block to an eviction
                                  //   committed within the kWindow requests before it
  // staging of the coming requests by the probe warps (kStageDepth stages + two of the route warp)
  volatile uint32_t* st_ready;    // [kStageDepth] request (+1) whose data the stage holds
  volatile uint32_t* st_pc;       // [kStageDepth] requests known committed before the masks were read
  uint32_t* st_hits;              // [kStages][R] prefix hits
  double* st_ab;                  // [kStages][R] (w_net*RTT + w_prefill*uncached) per replica
  uint32_t* st_ids;               // [kStages][kStageBlocks] block ids
  MaskT* st_mk;                   // [kStages][kStageBlocks] mask words
};

// Keeps the compiler from moving ordinary loads above the polling of a flag that guards them
// (the hardware issues a warp's shared-memory accesses in program order).
__device__ __forceinline__ void compiler_fence() { asm volatile("" ::: "memory"); }

// A warp that ran into a limit: record it and tell the other warps of the candidate to stop.
__device__ __forceinline__ void give_up(volatile uint32_t* ctl, int32_t status, uint32_t lane) {
  if (lane == 0) {
    atomicMin(const_cast<int32_t*>(reinterpret_cast<volatile int32_t*>(ctl + kCtlStatus)), status);
    ctl[kCtlAbort] = 1;
  }
}

// What a warp needs to know of a request ahead of time.
struct Ahead { uint32_t off, nblk, prev_share, in_tok, origin; };
__device__ __forceinline__ Ahead fetch_ahead(const ReqRec* req, uint32_t q, uint32_t end) {
  Ahead h = {0u, 0u, kNone, 0u, 0u};
  if (q < end) {
    const ReqRec x = req[q];
    h.off = x.off; h.nblk = x.nblk; h.prev_share = x.prev_share; h.in_tok = x.in_tok;
    h.origin = x.origin;
  }
  return h;
}

// Prefix probe on every replica from staged mask words: h_i = leading blocks whose mask has
// bit i.  The first kStageBlocks words come from `smk`; longer prompts read the rest from memory.
template <typename MaskT>
__device__ __forceinline__ void probe_staged(const MaskT* smk, const MaskT* mask,
                                             const uint32_t* ids, const Ahead& q, uint32_t R,
                                             uint32_t lane, uint32_t& h0, uint32_t& h1) {
  h0 = 0; h1 = 0;   // this lane's replicas: lane and lane+32
  const uint32_t n = q.nblk;
  MaskT alive = (R >= sizeof(MaskT) * 8) ? (MaskT)~(MaskT)0 : (MaskT)((((MaskT)1) << (R & 63)) - 1);
  for (uint32_t c = 0; c < n && alive != 0; c += 32) {
    const uint32_t k = c + lane;
    MaskT m = 0;
    if (k < n) m = (c < kStageBlocks) ? smk[k] : mask_load<MaskT>(mask, ids[q.off + k]);
    MaskT it = (MaskT)(shfl_mask<MaskT>(m, 0) & alive);
    MaskT still = 0;
    while (it != 0) {
      const int i = first_bit<MaskT>(it);
      it &= (MaskT)(it - 1);
      const unsigned b = __ballot_sync(kFull, (m >> i) & 1);
      const uint32_t run = (b == kFull) ? 32u : (uint32_t)__ffs((int)~b) - 1u;
      if ((uint32_t)(i & 31) == lane) {
        if (i < 32) h0 += run; else h1 += run;
      }
      if (run == 32u) still |= (MaskT)(((MaskT)1) << i);
    }
    alive = still;
  }
}

// Stage the prefix hits of a request and the part of its score (Eq. 3) that depends on them:
// ab_i = (w_net * RTT[g][i]) + (w_prefill * uncached_i), same operations and order as the score.
template <typename MaskT>
__device__ __forceinline__ void stage_scores(const ReplayArgs& a, const Ctx<MaskT>& cx,
                                             const Ahead& q, uint32_t slot, uint32_t h0,
                                             uint32_t h1, uint32_t lane) {
  const uint32_t R = a.m.R;
  const double w_pre = cx.sm.w[1];
  const double* wrtt_row = cx.sm.wrtt + (size_t)q.origin * R;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const uint32_t i = lane + 32u * half;
    if (i < R) {
      const uint32_t h = half ? h1 : h0;
      const unsigned long long hb = (unsigned long long)h * a.m.B;
      const uint32_t unc = q.in_tok - (uint32_t)(hb < q.in_tok ? hb : q.in_tok);
      cx.st_hits[slot * R + i] = h;
      cx.st_ab[slot * R + i] = __dadd_rn(wrtt_row[i], __dmul_rn(w_pre, (double)unc));
    }
  }
}

// Probe warp `which` of kProbeWarps: works on requests first+which, first+which+kProbeWarps, ...
// up to kWindow requests ahead of the cache warp.  For request q it reads the block ids and the
// mask words (first kStageBlocks blocks), stages them in shared memory, probes them and publishes
// the prefix hits together with the number of requests known to be committed when the masks
// were read.  Commits after that number may or may not show in the read; the route warp uses the
// stage only if none of them can have touched a block of q, else it repeats the probe itself,
// so results never depend on the timing of this warp, which may also stop at any time.
template <typename MaskT>
__device__ __forceinline__ void probe_warp(const ReplayArgs& a, const Ctx<MaskT>& cx,
                                           uint32_t lane, uint32_t which) {
  const Smem& sm = cx.sm;
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  const MaskT* mask = cx.mask;
  const uint32_t R = a.m.R;
  const uint32_t end = a.first + a.count;
  const uint32_t q0 = a.first + which;
  Ahead q_a = fetch_ahead(req, q0, end), q_n = fetch_ahead(req, q0 + kProbeWarps, end);
  Ahead q_b = q_a;
  uint32_t id_a[kRegChunks], id_n[kRegChunks], id_b[kRegChunks];
  MaskT m_a[kRegChunks], m_b[kRegChunks];
  uint32_t pc_a = 0, pc_b = 0;
#pragma unroll
  for (int c = 0; c < kRegChunks; ++c) {
    const uint32_t k = c * 32u + lane;
    id_a[c] = (k < q_a.nblk) ? ids[q_a.off + k] : 0u;
    id_n[c] = 0u; id_b[c] = 0u; m_a[c] = (MaskT)0; m_b[c] = (MaskT)0;
  }
  GORGO_PROF_DECL
  for (uint32_t qa = q0; qa < end + kProbeWarps; qa += kProbeWarps) {
    GORGO_PT(0)
    if (qa > q0) {
      // stage and probe this warp's previous request (its mask words were requested a round ago)
      const uint32_t qb = qa - kProbeWarps, slot = qb % kStageDepth;
      uint32_t* sid = cx.st_ids + slot * kStageBlocks;
      MaskT* smk = cx.st_mk + slot * kStageBlocks;
#pragma unroll
      for (int c = 0; c < kRegChunks; ++c) {
        const uint32_t k = c * 32u + lane;
        if (k < q_b.nblk) { sid[k] = id_b[c]; smk[k] = m_b[c]; }
      }
      __syncwarp();
      uint32_t h0, h1;
      probe_staged<MaskT>(smk, mask, ids, q_b, R, lane, h0, h1);
      stage_scores<MaskT>(a, cx, q_b, slot, h0, h1, lane);
      if (lane == 0) cx.st_pc[slot] = pc_b;
      __threadfence_block();                  // (no load of this warp is in flight here)
      __syncwarp();
      if (lane == 0) cx.st_ready[slot] = qb + 1;
    }
    GORGO_PT(1)
    if (qa < end) {
      // the stage of request qa is free, and its read at most kWindow commits old, once request
      // qa - kStageDepth is committed
      uint32_t polls = 0;
      uint32_t pc = *sm.progress;
      while ((int32_t)(pc - qa) <= -(int32_t)kStageDepth) {
        if (*sm.abort || ++polls > (1u << 22)) {           // bounded wait
          if (lane == 0) atomicAdd(const_cast<uint32_t*>(cx.ctl + kCtlProbeGone), 1u);
          return;
        }
        __nanosleep(20);
        pc = *sm.progress;
      }
      pc_a = pc;
      GORGO_PT(2)
#pragma unroll
      for (int c = 0; c < kRegChunks; ++c) {
        const uint32_t k = c * 32u + lane;
        m_a[c] = (k < q_a.nblk) ? mask_load<MaskT>(mask, id_a[c]) : (MaskT)0;
        id_n[c] = (k < q_n.nblk) ? ids[q_n.off + k] : 0u;     // ids of this warp's next request
      }
    }
    const Ahead q_nn = fetch_ahead(req, qa + 2 * kProbeWarps, end);
    q_b = q_a; q_a = q_n; q_n = q_nn;
    pc_b = pc_a;
#pragma unroll
    for (int c = 0; c < kRegChunks; ++c) { id_b[c] = id_a[c]; m_b[c] = m_a[c]; id_a[c] = id_n[c]; }
  }
  GORGO_PROF_FLUSH(7 + which)
}

// Route warp: the serial heart of a replay.  For request r it takes the staged prefix hits and
// hit-dependent score terms, applies the staged expiries to the in-flight token counts (kept in
// registers: lane i owns replicas i and i+32), adds the queue term of Eq. 3, takes the
// lowest-index argmin and publishes the route.  Everything else (service model, cache commit)
// happens behind it in other warps.  A stage is used only if no commit since its masks were read
// can have touched the request: no request since then shares a block with it (static field
// `prev_share`) and the cache warp has not flagged the request (a block evicted by one of the
// last kWindow commits occurs in it).  Otherwise the warp waits for the cache warp and probes
// the request itself.
template <typename MaskT>
__device__ __forceinline__ void route_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t lane) {
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R, K = a.m.K;
  const uint32_t end = a.first + a.count;
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  volatile uint32_t* ctl = cx.ctl;
  const double w_que = sm.w[2];
  const uint32_t i0 = lane, i1 = lane + 32u;
  const double nrm0 = (K != 3 && i0 < R) ? sm.w[3 + i0] : 1.0;
  const double nrm1 = (K != 3 && i1 < R) ? sm.w[3 + i1] : 1.0;
  long long ld0 = i0 < R ? sm.load[i0] : 0, ld1 = i1 < R ? sm.load[i1] : 0;
  int32_t status = 0;
  Ahead q0 = fetch_ahead(req, a.first, end), q1 = fetch_ahead(req, a.first + 1, end),
        q2 = fetch_ahead(req, a.first + 2, end);

  GORGO_PROF_DECL
  for (uint32_t r = a.first; r < end; ++r) {
    const Ahead q = q0;
    q0 = q1; q1 = q2;
    q2 = fetch_ahead(req, r + 3, end);                   // in flight while three requests run
    uint32_t slot = r % kStageDepth;

    // ---- wait: expiries of r staged, room in the route ring, every earlier commit checked,
    //      the stage of r filled (or no probe warp left to fill it)
    uint32_t polls = 0;
    bool staged = false;
    while (true) {
      uint32_t mexp = ctl[kCtlExp], mserved = ctl[kCtlServed];
#pragma unroll
      for (uint32_t w = 1; w < kQueueWarps; ++w) {
        mexp = min(mexp, ctl[kCtlExp + w]);
        mserved = min(mserved, ctl[kCtlServed + w]);
      }
      const uint32_t ck = ctl[kCtlChecked];
      const uint32_t sready = cx.st_ready[slot];
      const uint32_t gone = ctl[kCtlProbeGone];
      if (mexp > r && r - mserved < kRouteRing && ck >= r && (sready == r + 1 || gone)) {
        staged = sready == r + 1;
        break;
      }
      if (ctl[kCtlAbort] || ++polls > kSpinLimit) { status = -6; break; }
      __nanosleep(kPollNs);
#ifdef GORGO_PROF
      if (!(mexp > r)) GORGO_PC(8, 1) else if (!(r - mserved < kRouteRing)) GORGO_PC(9, 1)
      else if (!(ck >= r)) GORGO_PC(10, 1) else GORGO_PC(11, 1)
#endif
    }
    GORGO_PT(0)
    if (status) break;
    compiler_fence();
    if (staged) {
      const uint32_t spc = cx.st_pc[slot];
      staged = (q.prev_share == kNone || q.prev_share < spc) && cx.inval[r % kInvalRing] != r + 1;
    }
    if (!staged) {
      GORGO_PC(12, 1)
      // every earlier commit has to be in the masks before they are read here
      polls = 0;
      while (ctl[kCtlApplied] < r) {
        if (ctl[kCtlAbort] || ++polls > kSpinLimit) { status = -6; break; }
      }
      if (status) break;
      __threadfence_block();
      slot = kStageDepth + (r & 1u);
      uint32_t* sid = cx.st_ids + slot * kStageBlocks;
      MaskT* smk = cx.st_mk + slot * kStageBlocks;
#pragma unroll
      for (int c = 0; c < kRegChunks; ++c) {
        const uint32_t k = c * 32u + lane;
        if (k < q.nblk) { const uint32_t id = ids[q.off + k]; sid[k] = id; smk[k] = mask_load<MaskT>(cx.mask, id); }
      }
      __syncwarp();
      uint32_t h0, h1;
      probe_staged<MaskT>(smk, cx.mask, ids, q, R, lane, h0, h1);
      stage_scores<MaskT>(a, cx, q, slot, h0, h1, lane);
      __syncwarp();
    }

    GORGO_PT(1)
    // ---- queue signal (Eq. 2): requests that completed by the arrival of r stop counting
    const volatile long long* sub = cx.exp_sub + (size_t)(r % kExpRing) * R;
    if (i0 < R) ld0 -= sub[i0];
    if (i1 < R) ld1 -= sub[i1];

    // ---- score of Eq. 3 (fixed order, no FMA): the staged (w_net*RTT + w_prefill*uncached)
    //      plus the queue term; lowest-index argmin
    uint64_t best_k = ~0ull;
    uint32_t best_i = kNone;
    if (i0 < R) {
      double qv = (double)ld0;
      if (K != 3) qv = __dmul_rn(qv, nrm0);
      double c = __dadd_rn(cx.st_ab[slot * R + i0], __dmul_rn(w_que, qv));
      if (c != c) c = (i0 == 0) ? -d_inf() : d_inf();    // a NaN score wins only at index 0
      best_k = order_key(c); best_i = i0;
    }
    if (i1 < R) {
      double qv = (double)ld1;
      if (K != 3) qv = __dmul_rn(qv, nrm1);
      double c = __dadd_rn(cx.st_ab[slot * R + i1], __dmul_rn(w_que, qv));
      if (c != c) c = d_inf();
      const uint64_t ck = order_key(c);
      if (ck < best_k || best_i == kNone) { best_k = ck; best_i = i1; }
    }
    GORGO_PT(2)
    const uint32_t istar = warp_argmin_key(best_k, best_i);
    GORGO_PT(3)
    const uint32_t hstar = cx.st_hits[slot * R + istar];
    if (lane == 0) {
      cx.route_ring[r % kRouteRing] = istar | (slot << 8) | (hstar << 16);
      cx.route_log[r] = (uint8_t)istar;
    }
    __threadfence_block();
    __syncwarp();
    if (lane == 0) ctl[kCtlRouted] = r + 1;
    if ((istar & 31u) == lane) {
      if (istar < 32u) ld0 += (long long)q.in_tok; else ld1 += (long long)q.in_tok;
    }
    GORGO_PT(4)
  }
  GORGO_PROF_FLUSH(0)
  if (i0 < R) sm.load[i0] = ld0;
  if (i1 < R) sm.load[i1] = ld1;
  if (status != 0) give_up(ctl, status, lane);
}

// Queue warp `which` of kQueueWarps: owns the replicas i with i mod kQueueWarps == which.  It
// does two things, both in request order:
//  (A) books routed request j on its replica: earliest-free slot (lowest index on ties), start,
//      first-token and finish times, outputs; the request joins the slot's FIFO of in-flight
//      requests;
//  (B) stages, for a coming request e, the tokens that stop being in flight on each of its
//      replicas at the arrival of e (finish <= t'_e), for the route warp to subtract.
// (B) for e may run ahead of the routing: it only needs (A) done for the requests that can
// have finished by t'_e, which the static bound `need_svc[e]` gives (a request cannot finish
// before its arrival plus its decode time).  (A) for j runs after (B) for j, so (B) never sees
// a request that arrives later than e.
template <typename MaskT>
__device__ __forceinline__ void queue_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p,
                                           uint32_t lane, uint32_t which) {
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R, S = a.m.S;
  const uint32_t N = a.tr.n_req;
  const ReqRec* req = a.tr.req;
  double *free_at = cx.free_at, *q0_fin = cx.q0_fin, *q1_fin = cx.q1_fin;
  uint32_t *q0_tok = cx.q0_tok, *q1_tok = cx.q1_tok, *q2_idx = cx.q2_idx, *tail = cx.tail,
           *qcnt = cx.qcnt;
  uint4* qrec = cx.qrec;
  volatile uint32_t* ctl = cx.ctl;
  int32_t status = 0;
  unsigned long long st_hit = 0, st_blk = 0;
  const uint32_t end = a.first + a.count;
  const uint32_t last_r = end - 1;

  // a slot whose second-oldest entry has to be refilled from the per-request records: slot index
  // (kNone: none), record to read, whether the read has been issued, and the record read.  The
  // read is issued after the expiries are published, so that nothing waits for it.
  uint32_t pend_x = kNone, pend_idx = kNone;
  bool pend_loaded = false;
  uint4 pend_rec = make_uint4(0, 0, 0, 0);
  auto flush_pending = [&]() {
    if (pend_x != kNone) {
      if (!pend_loaded) pend_rec = qrec[pend_idx];
      q1_fin[pend_x] = __hiloint2double((int)pend_rec.y, (int)pend_rec.x);
      q2_idx[pend_x] = pend_rec.z;
      q1_tok[pend_x] = pend_rec.w;
      pend_x = kNone;
    }
  };

  uint32_t ja = a.first, e = a.first;
  // static data of the coming requests, fetched two ahead of each cursor
  ReqRec ra0 = req[min(ja, last_r)], ra1 = req[min(ja + 1, last_r)];
  double te0 = a.tq[min(e, last_r)], te1 = a.tq[min(e + 1, last_r)];
  uint32_t nd0 = a.need_svc[min(e, last_r)], nd1 = a.need_svc[min(e + 1, last_r)];
  uint32_t idle = 0;

  GORGO_PROF_DECL
  while (ja < end || e < end) {
    const uint32_t routed = ctl[kCtlRouted];
    GORGO_PT(0)
    if (e < end && e < routed + kExpRing && ja >= nd0) {
      // ---- (B) expiries at the arrival of request e
      const double t = te0;                        // = scale * ts[e]
      long long* sub = cx.exp_sub + (size_t)(e % kExpRing) * R;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint32_t i = lane + 32u * half;
        if (i < R && (i % kQueueWarps) == which) sub[i] = 0;
      }
      __syncwarp();
      for (uint32_t i0 = 0; i0 < R; i0 += 32) {
        const uint32_t i = i0 + lane;
        unsigned due = __ballot_sync(kFull, i < R && (i % kQueueWarps) == which && sm.minfin[i] <= t);
        while (due) {
          const uint32_t ii = i0 + (uint32_t)__ffs((int)due) - 1;
          due &= due - 1;
          long long tok = 0;
          double mn = d_inf();
          for (uint32_t s = lane; s < S; s += 32) {
            const uint32_t x = ii * S + s;
            double hf = q0_fin[x];
            if (hf <= t) {
              uint32_t guard = 0;
              uint32_t cnt = qcnt[x];
              do {
                if (pend_x == x) flush_pending();           // the second entry is still in flight
                tok += (long long)q0_tok[x];
                --cnt;
                if (cnt == 0) { hf = d_inf(); }
                else {
                  hf = q1_fin[x];                            // the second becomes the oldest
                  q0_tok[x] = q1_tok[x];
                  if (cnt >= 2) {                            // the new second is fetched later
                    flush_pending();
                    pend_x = x;
                    pend_idx = q2_idx[x];
                    pend_loaded = false;
                  }
                }
                if (++guard > N) { status = -6; break; }
              } while (hf <= t);
              q0_fin[x] = hf;
              qcnt[x] = cnt;
            }
            mn = fmin(mn, hf);
          }
          if (tok != 0)
            atomicAdd(reinterpret_cast<unsigned long long*>(sub + ii), (unsigned long long)tok);
          uint64_t mk = order_key(mn);
          warp_argmin_key(mk, lane);
          if (lane == 0) sm.minfin[ii] = order_value(mk);
        }
      }
      __threadfence_block();
      __syncwarp();
      if (lane == 0) ctl[kCtlExp + which] = e + 1;
      if (pend_x != kNone && !pend_loaded) { pend_rec = qrec[pend_idx]; pend_loaded = true; }
      ++e;
      te0 = te1; nd0 = nd1;
      te1 = a.tq[min(e + 1, last_r)];
      nd1 = a.need_svc[min(e + 1, last_r)];
      idle = 0;
      GORGO_PT(1)
      if (__any_sync(kFull, status != 0)) break;
      continue;
    }
    if (ja < routed && ja < e) {
      // ---- (A) service commit of routed request ja, if its replica is one of this warp's
      const uint32_t ent = cx.route_ring[ja % kRouteRing];
      const uint32_t istar = ent & 255u, hstar = ent >> 16;
      if ((istar % kQueueWarps) == which) {
        const ReqRec rec = ra0;
        const uint32_t r = ja, in_tok = rec.in_tok;
        const double t = __dmul_rn(a.scale, rec.ts_ms);
        const unsigned long long hbstar = (unsigned long long)hstar * a.m.B;
        const uint32_t uncstar = in_tok - (uint32_t)(hbstar < in_tok ? hbstar : in_tok);
        // earliest-free slot, lowest index on ties
        uint64_t bk = ~0ull;
        uint32_t bs = kNone;
        for (uint32_t s = lane; s < S; s += 32) {
          const uint64_t vk = order_key(free_at[(size_t)istar * S + s]);
          if (vk < bk || bs == kNone) { bk = vk; bs = s; }
        }
        bs = warp_argmin_key(bk, bs);
        const double bv = order_value(bk);
        const double arrive = __dadd_rn(t, sm.rtt[(size_t)rec.origin * R + istar]);
        const double start = (bv > arrive) ? bv : arrive;
        const double first = __dadd_rn(start, __dmul_rn(a.m.prefill_ms, (double)uncstar));
        const uint32_t dec_tok = rec.out_tok > 0 ? rec.out_tok - 1 : 0;
        const double finish = __dadd_rn(first, __dmul_rn(a.m.tpot_ms, (double)dec_tok));
        if (pend_x == istar * S + bs) flush_pending();   // the slot's own refill comes first
        __syncwarp();
        if (lane == 0) {
          const size_t x = (size_t)istar * S + bs;
          qrec[r] = make_uint4((uint32_t)__double2loint(finish), (uint32_t)__double2hiint(finish),
                               kNone, in_tok);
          const uint32_t cnt = qcnt[x];
          if (cnt == 0) {
            q0_fin[x] = finish; q0_tok[x] = in_tok;
            sm.minfin[istar] = fmin(sm.minfin[istar], finish);
          } else {
            reinterpret_cast<uint32_t*>(qrec + tail[x])[2] = r;     // link behind the newest
            if (cnt == 1) { q1_fin[x] = finish; q1_tok[x] = in_tok; q2_idx[x] = kNone; }
            else if (cnt == 2) q2_idx[x] = r;
          }
          qcnt[x] = cnt + 1;
          tail[x] = r;
          free_at[x] = finish;
          const size_t o = (size_t)p * a.out_stride + (r - a.first);
          if (a.route_out) a.route_out[o] = (uint8_t)istar;
          if (a.hit_out) a.hit_out[o] = (uint16_t)hstar;
          if (a.ttft_out) a.ttft_out[o] = __dsub_rn(first, t);
          if (a.e2e_out) a.e2e_out[o] = __dsub_rn(finish, t);
          st_hit += hstar; st_blk += rec.nblk;
        }
        __syncwarp();
      }
      ++ja;
      ra0 = ra1;
      ra1 = req[min(ja + 1, last_r)];
      if (lane == 0) ctl[kCtlServed + which] = ja;
      idle = 0;
#ifdef GORGO_PROF
      if ((istar % kQueueWarps) == which) GORGO_PT(2) else GORGO_PT(3)
#endif
      continue;
    }
    if (ctl[kCtlAbort] || ++idle > kSpinLimit) { status = -6; break; }
    __nanosleep(2 * kPollNs);
  }
  GORGO_PROF_FLUSH(3 + which)
  flush_pending();
  __syncwarp();
  status = __reduce_min_sync(kFull, status);
  if (status != 0) give_up(ctl, status, lane);
  if (lane == 0 && a.stats) {
    unsigned long long* s4 = reinterpret_cast<unsigned long long*>(a.stats) + (size_t)p * 4;
    atomicAdd(s4 + 1, st_hit);
    atomicAdd(s4 + 2, st_blk);
  }
}

// The cache commit of a routed request is split between two warps.
//
// Check warp (on the serial path): from the staged mask words of request r it counts the blocks
// missing on the chosen replica, sizes the eviction and takes the victims from the head of the
// replica's ring.  A victim whose block occurs again in one of the next kWindow requests voids
// that request's staged read: the request is flagged before the route warp is told that the
// victims of r are known, which is all the route warp waits for.  In the common case this warp
// touches shared memory only; the memory traffic of the commit is left to the apply warp as a
// work item.  If the ring cannot serve the eviction as it stands (the scout is behind, or an
// entry went stale), the warp waits until every earlier commit is applied and evicts by the
// general procedure itself.
//
// Apply warp (behind): sets the replica's bit on the missing blocks, clears it on the victims,
// appends the request to the replica's recency list and publishes the request as committed.
struct ApplyItem {
  uint32_t route;     // replica | stage << 8
  uint32_t head0;     // ring index of the first victim left to this warp
  uint32_t nvict;     // victims left to this warp (0: the check warp evicted itself)
  uint32_t evicted;   // victims of the request in all (statistics)
  uint32_t lru_prev;  // previous request routed to the replica (kNone: none)
  uint32_t nblk, off, pad;
};

template <typename MaskT>
__device__ __forceinline__ void check_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t lane) {
  const Smem& sm = cx.sm;
  const uint32_t N = a.tr.n_req;
  const ReqRec* req = a.tr.req;
  const uint32_t* ids = a.tr.ids;
  MaskT* mask = cx.mask;
  uint32_t* lru_next = cx.lru_next;
  const uint8_t* route_log = cx.route_log;
  volatile uint32_t* ctl = cx.ctl;
  int32_t status = 0;
  const unsigned long long evict_guard_max = (unsigned long long)N + a.tr.n_ids / 16u + 64u;
  const uint32_t end = a.first + a.count;

  Ahead q_cur = fetch_ahead(req, a.first, end), q_nxt = fetch_ahead(req, a.first + 1, end);

  GORGO_PROF_DECL
  for (uint32_t r = a.first; r < end; ++r) {
    const uint32_t n = q_cur.nblk, off = q_cur.off;
    const Ahead q_n2 = fetch_ahead(req, r + 2, end);          // used two rounds from now

    // ---- wait for the route of request r (and for room in the apply ring)
    uint32_t polls = 0;
    while (ctl[kCtlRouted] <= r || r - ctl[kCtlApplied] >= kApplyRing) {
      if (ctl[kCtlAbort] || ++polls > kSpinLimit) { status = -6; break; }
      __nanosleep(kPollNs);
    }
    GORGO_PT(0)
    if (status) break;
    compiler_fence();
    const uint32_t ent0 = cx.route_ring[r % kRouteRing];
    const uint32_t istar = ent0 & 255u, slot = (ent0 >> 8) & 255u;
    const MaskT bit = (MaskT)(((MaskT)1) << istar);
    const MaskT* smk = cx.st_mk + slot * kStageBlocks;
    GORGO_PT(6)

    // ---- blocks of r missing on the replica
    uint32_t missing = 0;
#pragma unroll
    for (int c = 0; c < kRegChunks; ++c) {
      if ((uint32_t)c * 32u < n) {
        const uint32_t k = (uint32_t)c * 32u + lane;
        const bool miss = k < n && !(smk[k] & bit);
        missing += __popc(__ballot_sync(kFull, miss));
      }
    }
    for (uint32_t c = kStageBlocks; c < n; c += 32) {      // longer prompts: the rest from memory
      const uint32_t k = c + lane;
      const bool miss = k < n && !(mask_load<MaskT>(mask, ids[off + k]) & bit);
      missing += __popc(__ballot_sync(kFull, miss));
    }
    GORGO_PT(1)
    uint32_t occ = sm.occ[istar] + missing;
    uint32_t need = occ > a.m.C ? (uint32_t)(occ - a.m.C) : 0u;
    uint32_t evicted = 0, nvict = 0;
    GORGO_PC(9, n) GORGO_PC(10, need)
    const uint32_t head0 = sm.chead[istar];
    if (need > 0) {
      uint32_t cr = sm.curreq[istar];
      int32_t cp = sm.curpos[istar];
      const uint4* lst = sm.lst + (size_t)istar * kListCap;
      // ---- common case: the next `need` ring entries are all live; they are the victims
      bool clean = sm.act[istar] != 0;
      if (clean) {
        uint32_t avail = sm.ring_tail[istar] - head0;
        for (uint32_t polls2 = 0; avail < need && polls2 < 64; ++polls2) {
          __nanosleep(20);
          avail = sm.ring_tail[istar] - head0;
          GORGO_PC(11, 1)
        }
        clean = avail >= need;
        compiler_fence();
      }
      GORGO_PT(4)
      uint32_t last_w = 0, last_z = 0;
      for (uint32_t o = 0; clean && o < need; o += 32) {
        const bool mine = o + lane < need;
        uint4 ent = make_uint4(0, kNone, 0, 0);
        bool odd = false;        // void (behind the cursor) or touched again since it was listed
        if (mine) {
          const uint32_t e = (head0 + o + lane) & (kListCap - 1);
          ent = a.lists_in_smem ? lst[e] : __ldcg(lst + e);
          odd = ent.y <= r || ent.w < cr || (ent.w == cr && (int32_t)ent.z > cp);
        }
        if (__any_sync(kFull, odd)) { clean = false; break; }
        // a victim that occurs again within the window voids that request's staged read
        const bool soon = mine && ent.y - (r + 1) < kWindow;
        if (__any_sync(kFull, soon)) {
          if (soon) cx.inval[ent.y % kInvalRing] = ent.y + 1;
          __threadfence_block();
        }
        const uint32_t lastl = min(need - o, 32u) - 1u;   // lane of the last victim of the round
        last_w = __shfl_sync(kFull, ent.w, lastl);
        last_z = __shfl_sync(kFull, ent.z, lastl);
      }
      GORGO_PT(5)
      if (clean) {
        cr = last_w;
        cp = (int32_t)last_z - 1;
        evicted = nvict = need;
        need = 0;
        if (lane == 0) sm.chead[istar] = head0 + nvict;
      } else {
        GORGO_PC(8, 1)
        // ---- general procedure, by this warp, once every earlier commit is applied
        polls = 0;
        while (ctl[kCtlApplied] < r) {
          if (ctl[kCtlAbort] || ++polls > kSpinLimit) { status = -6; break; }
        }
        if (status) break;
        __threadfence_block();
        if (sm.act[istar]) {
          uint32_t head = head0;     // == ring_head: the apply warp has caught up
          uint32_t last_e = kNone;   // ring slot of the last entry passed that was not void
          while (need > 0) {
            uint32_t avail = sm.ring_tail[istar] - head;
            for (uint32_t polls2 = 0; avail == 0 && polls2 < 64; ++polls2) {
              __nanosleep(20);
              avail = sm.ring_tail[istar] - head;
            }
            if (avail == 0) break;                          // the scout is behind: walk ourselves
            const uint32_t m = min(avail, 32u);
            uint4 ent = make_uint4(0, kNone, 0, 0);
            bool live = false;
            uint32_t nxr = kNone;      // request of the block's next occurrence after r
            if (lane < m) {
              const uint32_t e = (head + lane) & (kListCap - 1);
              ent = a.lists_in_smem ? lst[e] : __ldcg(lst + e);
              nxr = ent.y;
              // entries the eviction cursor has already passed (after a walk of our own) are void
              live = !(ent.w < cr || (ent.w == cr && (int32_t)ent.z > cp));
              if (live && ent.y <= r) {
                // the block came back since the entry was made: follow its occurrences up to r
                uint2 c = a.tr.occ_next[req[ent.w].off + ent.z];
                nxr = kNone;
                while (c.x != kNone) {
                  if (c.y > r) { nxr = c.y; break; }
                  const uint32_t rr = (c.y == r) ? istar : (uint32_t)route_log[c.y];
                  if (rr == istar) { live = false; break; }
                  c = a.tr.occ_next[c.x];
                }
              }
            }
            const unsigned lv = __ballot_sync(kFull, live);
            const uint32_t cnt = __popc(lv);
            const bool mine = live && (uint32_t)__popc(lv & ((1u << lane) - 1u)) < need;
            if (mine) mask_clear_bit<MaskT>(mask, ent.x, bit);
            {
              const bool soon = mine && nxr - (r + 1) < kWindow;
              if (__any_sync(kFull, soon)) {
                if (soon) cx.inval[nxr % kInvalRing] = nxr + 1;
                __threadfence_block();
              }
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
          if (lane == 0) { sm.chead[istar] = head; sm.ring_head[istar] = head; }
        }
        uint32_t coff = (cr != kNone && need > 0) ? req[cr].off : 0u;
        unsigned long long guard = 0;
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
          if (mine) mask_clear_bit<MaskT>(mask, vid, bit);
          {
            const bool soon = mine && nxr - (r + 1) < kWindow;
            if (__any_sync(kFull, soon)) {
              if (soon) cx.inval[nxr % kInvalRing] = nxr + 1;
              __threadfence_block();
            }
          }
          cp -= (cnt <= need) ? 32 : 32 - __clz((int)take);
          const uint32_t tk = __popc(take);
          need -= tk;
          evicted += tk;
        }
        __threadfence_block();                            // this warp's own reductions
      }
      if (lane == 0) { sm.curreq[istar] = cr; sm.curpos[istar] = cp; }
    }
    occ -= evicted;

    // ---- the victims of r are known: the route warp may go on
    __syncwarp();
    if (lane == 0) ctl[kCtlChecked] = r + 1;
    GORGO_PT(2)

    // ---- hand the memory traffic of the commit to the apply warp
    if (lane == 0) {
      sm.occ[istar] = occ;
      const uint32_t lt = sm.c_lrutail[istar];
      sm.c_lrutail[istar] = r;
      if (sm.curreq[istar] == kNone) { sm.curreq[istar] = r; sm.curpos[istar] = (int32_t)n - 1; }
      // hand the replica to the scout warp once its cache is close to full (before that no
      // eviction has happened here, so the scout starts from the eviction cursor)
      if (!sm.act[istar] && (uint64_t)occ + kPostMargin >= a.m.C) {
        sm.scan_cr[istar] = sm.curreq[istar];
        sm.scan_cp[istar] = sm.curpos[istar];
        __threadfence_block();
        sm.act[istar] = 1;
      }
      uint4* item = cx.apply_ring + (size_t)(r % kApplyRing) * 2;
      item[0] = make_uint4(istar | (slot << 8), head0, nvict, evicted);
      item[1] = make_uint4(lt, n, off, 0u);
      __threadfence_block();
      ctl[kCtlEnqueued] = r + 1;
    }
    __syncwarp();
    if (__any_sync(kFull, status != 0)) break;
    GORGO_PT(3)

    q_cur = q_nxt; q_nxt = q_n2;
  }
  GORGO_PROF_FLUSH(1)
  status = __reduce_min_sync(kFull, status);
  if (status != 0) give_up(ctl, status, lane);
}

template <typename MaskT>
__device__ __forceinline__ void apply_warp(const ReplayArgs& a, const Ctx<MaskT>& cx, uint32_t p,
                                           uint32_t lane) {
  const Smem& sm = cx.sm;
  const uint32_t R = a.m.R;
  const uint32_t* ids = a.tr.ids;
  MaskT* mask = cx.mask;
  uint32_t* lru_next = cx.lru_next;
  volatile uint32_t* ctl = cx.ctl;
  int32_t status = 0;
  unsigned long long st_probe = 0, st_evict = 0;
  const uint32_t end = a.first + a.count;

  GORGO_PROF_DECL
  for (uint32_t r = a.first; r < end; ++r) {
    uint32_t polls = 0;
    while (ctl[kCtlEnqueued] <= r) {
      if (ctl[kCtlAbort] || ++polls > kSpinLimit) { status = -6; break; }
      __nanosleep(20);
    }
    GORGO_PT(0)
    if (status) break;
    compiler_fence();
    const uint4* item = cx.apply_ring + (size_t)(r % kApplyRing) * 2;
    const uint4 i0 = item[0], i1 = item[1];
    const uint32_t istar = i0.x & 255u, slot = (i0.x >> 8) & 255u;
    const uint32_t head0 = i0.y, nvict = i0.z, n = i1.y, off = i1.z;
    const MaskT bit = (MaskT)(((MaskT)1) << istar);
    const uint32_t* sid = cx.st_ids + slot * kStageBlocks;
    const MaskT* smk = cx.st_mk + slot * kStageBlocks;

    // ---- set the replica's bit on the missing blocks
    for (uint32_t c = 0; c < n; c += 32) {
      const uint32_t k = c + lane;
      if (k < n) {
        uint32_t id;
        MaskT mv;
        if (c < kStageBlocks) { id = sid[k]; mv = smk[k]; }
        else { id = ids[off + k]; mv = mask_load<MaskT>(mask, id); }
        if (!(mv & bit)) mask_store<MaskT>(mask, id, (MaskT)(mv | bit));
      }
    }
    GORGO_PT(1)
    // ---- clear it on the victims the check warp took from the ring
    const uint4* lst = sm.lst + (size_t)istar * kListCap;
    for (uint32_t o = lane; o < nvict; o += 32) {
      const uint32_t e = (head0 + o) & (kListCap - 1);
      const uint4 ent = a.lists_in_smem ? lst[e] : __ldcg(lst + e);
      mask_clear_bit<MaskT>(mask, ent.x, bit);
    }
    if (lane < R) { const uint32_t h = cx.st_hits[slot * R + lane]; st_probe += (h + 1 < n ? h + 1 : n); }
    if (lane + 32u < R) { const uint32_t h = cx.st_hits[slot * R + lane + 32u]; st_probe += (h + 1 < n ? h + 1 : n); }
    st_evict += i0.w;
    if (lane == 0) {
      // recency order of the replica: append this request
      if (i1.x != kNone) lru_next[i1.x] = r;
      lru_next[r] = kNone;
    }
    GORGO_PT(2)
    __threadfence_block();                                // every lane's stores and reductions
    __syncwarp();
    GORGO_PT(3)
    if (lane == 0) {
      sm.lrutail[istar] = r;
      if (nvict) sm.ring_head[istar] = head0 + nvict;     // the scout may reuse these entries
      ctl[kCtlApplied] = r + 1;                           // request r is fully committed
    }
    __syncwarp();
    GORGO_PT(4)
  }
  GORGO_PROF_FLUSH(2)
  st_probe = warp_sum_u64(st_probe);
  if (status != 0) give_up(ctl, status, lane);
  if (lane == 0 && a.stats) {
    unsigned long long* s4 = reinterpret_cast<unsigned long long*>(a.stats) + (size_t)p * 4;
    atomicAdd(s4 + 0, st_probe);
    atomicAdd(s4 + 3, st_evict);
  }
}

constexpr uint32_t kWarpRoute = 0, kWarpCheck = 1, kWarpApply = 2, kWarpQueue0 = 3,
                   kWarpProbe0 = kWarpQueue0 + kQueueWarps, kWarpScout0 = kWarpProbe0 + kProbeWarps;
constexpr uint32_t kReplayThreads = 32 * (kWarpScout0 + kScouts);

// Byte offsets of the regions of a replay CTA's dynamic shared memory.
struct SmemPlan {
  uint32_t rtt, wrtt, w, minfin, load, slot_d, exp_sub, st_ab, ctl, occ, curreq, curpos, lrutail,
      slot_u, act, ring_head, ring_tail, scan_cr, scan_cp, c_lrutail, chead, route_ring, inval,
      apply_ring, st_ready, st_pc, st_hits,
      st_ids, st_mk, lst, total;
};
__host__ __device__ inline SmemPlan smem_plan(uint32_t R, uint32_t G, uint32_t S, uint32_t K,
                                              uint32_t mask_bytes, bool slots_in_smem,
                                              bool lists_in_smem) {
  SmemPlan p;
  uint32_t o = 0;
  const uint32_t RS = R * S;
#define GORGO_TAKE(field, bytes, align) \
  o = (o + (align) - 1u) / (align) * (align); p.field = o; o += (uint32_t)(bytes);
  GORGO_TAKE(rtt, G * R * 8u, 16u)
  GORGO_TAKE(wrtt, G * R * 8u, 8u)
  GORGO_TAKE(w, K * 8u, 8u)
  GORGO_TAKE(minfin, R * 8u, 8u)
  GORGO_TAKE(load, R * 8u, 8u)
  GORGO_TAKE(slot_d, slots_in_smem ? 3u * RS * 8u : 0u, 8u)
  GORGO_TAKE(exp_sub, kExpRing * R * 8u, 8u)
  GORGO_TAKE(st_ab, kStages * R * 8u, 8u)
  GORGO_TAKE(ctl, kCtlWords * 4u, 8u)
  GORGO_TAKE(occ, R * 4u, 4u)
  GORGO_TAKE(curreq, R * 4u, 4u)
  GORGO_TAKE(curpos, R * 4u, 4u)
  GORGO_TAKE(lrutail, R * 4u, 4u)
  GORGO_TAKE(slot_u, slots_in_smem ? 5u * RS * 4u : 0u, 4u)
  GORGO_TAKE(act, R * 4u, 4u)
  GORGO_TAKE(ring_head, R * 4u, 4u)
  GORGO_TAKE(ring_tail, R * 4u, 4u)
  GORGO_TAKE(scan_cr, R * 4u, 4u)
  GORGO_TAKE(scan_cp, R * 4u, 4u)
  GORGO_TAKE(c_lrutail, R * 4u, 4u)
  GORGO_TAKE(chead, R * 4u, 4u)
  GORGO_TAKE(route_ring, kRouteRing * 4u, 4u)
  GORGO_TAKE(inval, kInvalRing * 4u, 4u)
  GORGO_TAKE(st_ready, kStageDepth * 4u, 4u)
  GORGO_TAKE(st_pc, kStageDepth * 4u, 4u)
  GORGO_TAKE(st_hits, kStages * R * 4u, 4u)
  GORGO_TAKE(st_ids, kStages * kStageBlocks * 4u, 4u)
  GORGO_TAKE(st_mk, kStages * kStageBlocks * mask_bytes, 8u)
  GORGO_TAKE(apply_ring, kApplyRing * 32u, 16u)
  GORGO_TAKE(lst, lists_in_smem ? R * kListCap * 16u : 0u, 16u)
#undef GORGO_TAKE
  p.total = (o + 15u) / 16u * 16u;
  return p;
}

template <typename MaskT>
__global__ void __launch_bounds__(kReplayThreads, 2) replay_kernel(const ReplayArgs a) {
  const uint32_t p = blockIdx.x;
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t R = a.m.R, S = a.m.S, K = a.m.K, G = a.m.G;
  const uint32_t N = a.tr.n_req;
  const uint32_t RS = R * S;

  unsigned char* st = a.states + (size_t)p * a.lay.bytes;
  CandHeader* hdr = reinterpret_cast<CandHeader*>(st);
  RepState* g_rep = reinterpret_cast<RepState*>(st + a.lay.rep_off);
  double* g_slot_d = reinterpret_cast<double*>(st + a.lay.slot_d_off);     // 3 x [R*S] doubles
  uint32_t* g_slot_u = reinterpret_cast<uint32_t*>(st + a.lay.slot_u_off);  // 5 x [R*S] words

  extern __shared__ __align__(16) unsigned char smem_raw[];
  const SmemPlan pl = smem_plan(R, G, S, K, (uint32_t)sizeof(MaskT), a.slots_in_smem != 0,
                                a.lists_in_smem != 0);
  Ctx<MaskT> cx;
  Smem& sm = cx.sm;
  sm.rtt = reinterpret_cast<double*>(smem_raw + pl.rtt);        // [G*R]
  sm.wrtt = reinterpret_cast<double*>(smem_raw + pl.wrtt);      // [G*R]  w_net * rtt
  sm.w = reinterpret_cast<double*>(smem_raw + pl.w);            // [K]
  sm.minfin = reinterpret_cast<double*>(smem_raw + pl.minfin);  // [R]
  sm.load = reinterpret_cast<long long*>(smem_raw + pl.load);   // [R]
  // Per-slot state (in shared memory when it fits, else it stays in global memory).  A slot is a
  // FIFO of in-flight requests whose finish times never decrease; its two oldest entries are
  // kept here, the rest is reached through the per-request records in global memory.
  double* slot_d = a.slots_in_smem ? reinterpret_cast<double*>(smem_raw + pl.slot_d) : g_slot_d;
  uint32_t* slot_u = a.slots_in_smem ? reinterpret_cast<uint32_t*>(smem_raw + pl.slot_u) : g_slot_u;
  cx.free_at = slot_d;                   // time the slot frees (finish of its newest request)
  cx.q0_fin = slot_d + RS;               // finish of the oldest in-flight request (+inf: none)
  cx.q1_fin = slot_d + 2 * (size_t)RS;   // finish of the second oldest
  cx.q0_tok = slot_u;                    // input tokens of the oldest
  cx.q1_tok = slot_u + RS;               //   and of the second oldest
  cx.q2_idx = slot_u + 2 * (size_t)RS;   // request index of the third oldest (kNone: none)
  cx.tail = slot_u + 3 * (size_t)RS;     // newest request queued on the slot
  cx.qcnt = slot_u + 4 * (size_t)RS;     // requests in flight on the slot
  cx.exp_sub = reinterpret_cast<long long*>(smem_raw + pl.exp_sub);
  cx.st_ab = reinterpret_cast<double*>(smem_raw + pl.st_ab);
  cx.ctl = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.ctl);
  sm.progress = cx.ctl + kCtlApplied;
  sm.abort = cx.ctl + kCtlAbort;
  sm.occ = reinterpret_cast<uint32_t*>(smem_raw + pl.occ);
  sm.curreq = reinterpret_cast<uint32_t*>(smem_raw + pl.curreq);
  sm.curpos = reinterpret_cast<int32_t*>(smem_raw + pl.curpos);
  sm.lrutail = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.lrutail);
  sm.c_lrutail = reinterpret_cast<uint32_t*>(smem_raw + pl.c_lrutail);
  sm.chead = reinterpret_cast<uint32_t*>(smem_raw + pl.chead);
  sm.act = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.act);
  sm.ring_head = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.ring_head);
  sm.ring_tail = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.ring_tail);
  sm.scan_cr = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.scan_cr);
  sm.scan_cp = reinterpret_cast<volatile int32_t*>(smem_raw + pl.scan_cp);
  cx.route_ring = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.route_ring);
  cx.inval = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.inval);
  cx.apply_ring = reinterpret_cast<uint4*>(smem_raw + pl.apply_ring);
  cx.st_ready = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.st_ready);
  cx.st_pc = reinterpret_cast<volatile uint32_t*>(smem_raw + pl.st_pc);
  cx.st_hits = reinterpret_cast<uint32_t*>(smem_raw + pl.st_hits);
  cx.st_ids = reinterpret_cast<uint32_t*>(smem_raw + pl.st_ids);
  cx.st_mk = reinterpret_cast<MaskT*>(smem_raw + pl.st_mk);
  sm.lst = a.lists_in_smem ? reinterpret_cast<uint4*>(smem_raw + pl.lst)
                           : a.evict_lists + (size_t)p * R * kListCap;
  cx.mask = reinterpret_cast<MaskT*>(a.masks + (size_t)p * a.mask_stride);
  cx.qrec = a.qrec + (size_t)p * N;   // per request: (finish lo, finish hi, next on slot, tokens)
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
    sm.minfin[i] = rs.min_fin; sm.load[i] = rs.load; sm.occ[i] = rs.occ;
    sm.curreq[i] = rs.cur_req; sm.curpos[i] = rs.cur_pos; sm.lrutail[i] = rs.lru_tail;
    sm.c_lrutail[i] = rs.lru_tail; sm.chead[i] = 0;
    sm.act[i] = 0; sm.ring_head[i] = 0; sm.ring_tail[i] = 0;
  }
  if (a.slots_in_smem) {
    for (uint32_t x = threadIdx.x; x < 3 * RS; x += blockDim.x) slot_d[x] = g_slot_d[x];
    for (uint32_t x = threadIdx.x; x < 5 * RS; x += blockDim.x) slot_u[x] = g_slot_u[x];
  }
  if (threadIdx.x < kCtlWords) {
    uint32_t v = 0;
    if (threadIdx.x == kCtlRouted || threadIdx.x == kCtlApplied || threadIdx.x == kCtlChecked ||
        threadIdx.x == kCtlEnqueued ||
        (threadIdx.x >= kCtlExp && threadIdx.x < kCtlServed + kQueueWarps))
      v = a.first;
    cx.ctl[threadIdx.x] = v;
  }
  if (threadIdx.x < kStageDepth) { cx.st_ready[threadIdx.x] = 0; cx.st_pc[threadIdx.x] = 0; }
  if (threadIdx.x < kInvalRing) cx.inval[threadIdx.x] = 0;
  __syncthreads();

  if (warp == kWarpRoute) route_warp<MaskT>(a, cx, lane);
  else if (warp == kWarpCheck) check_warp<MaskT>(a, cx, lane);
  else if (warp == kWarpApply) apply_warp<MaskT>(a, cx, p, lane);
  else if (warp < kWarpProbe0) queue_warp<MaskT>(a, cx, p, lane, warp - kWarpQueue0);
  else if (warp < kWarpScout0) probe_warp<MaskT>(a, cx, lane, warp - kWarpProbe0);
  else scout_warp<MaskT>(a, sm, cx.lru_next, cx.route_log, lane, warp - kWarpScout0);
  __syncthreads();

  // ---- write the small state back
  for (uint32_t i = threadIdx.x; i < R; i += blockDim.x) {
    RepState rs;
    rs.min_fin = sm.minfin[i]; rs.load = sm.load[i]; rs.occ = sm.occ[i];
    rs.cur_req = sm.curreq[i]; rs.cur_pos = sm.curpos[i]; rs.lru_tail = sm.lrutail[i];
    g_rep[i] = rs;
  }
  if (a.slots_in_smem) {
    for (uint32_t x = threadIdx.x; x < 3 * RS; x += blockDim.x) g_slot_d[x] = slot_d[x];
    for (uint32_t x = threadIdx.x; x < 5 * RS; x += blockDim.x) g_slot_u[x] = slot_u[x];
  }
  if (threadIdx.x == 0) {
    const int32_t status = (int32_t)cx.ctl[kCtlStatus];
    hdr->processed = a.first + a.count;
    if (status != 0) hdr->status = status;
    if (a.status_out && (status != 0 || !a.check_order)) a.status_out[p] = status;
  }
}

// ---------------------------------------------------------------- expiry lower bound
// need_svc[e] = one past the last request j < e (within the launch) that can have finished by
// the arrival of e.  A request finishes no earlier than its arrival plus its decode time
// (network, queueing and prefill only add to that, and every rounding is monotone), so with
// lb_j = t'_j + tpot * max(out_j - 1, 0) and e_j = first request after j with t'_e >= lb_j,
// need_svc[e] = max{ j + 1 : e_j <= e }.  Depends on the trace and the time scale only.
__global__ void need_scatter_kernel(const ReqRec* req, double scale, double tpot_ms,
                                    uint32_t first, uint32_t count, uint32_t* need, double* tq) {
  const uint32_t x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= count) return;
  const uint32_t j = first + x, end = first + count;
  const ReqRec rec = req[j];
  const uint32_t dec_tok = rec.out_tok > 0 ? rec.out_tok - 1 : 0;
  const double t = __dmul_rn(scale, rec.ts_ms);          // scaled arrival, kept for the queue warps
  tq[j] = t;
  const double lb = __dadd_rn(t, __dmul_rn(tpot_ms, (double)dec_tok));
  uint32_t lo = j + 1, hi = end;
  while (lo < hi) {
    const uint32_t mid = lo + (hi - lo) / 2;
    if (__dmul_rn(scale, req[mid].ts_ms) >= lb) hi = mid; else lo = mid + 1;
  }
  if (lo < end) atomicMax(need + lo, j + 1);
}

constexpr int kScanThreads = 1024;
__global__ void __launch_bounds__(kScanThreads) need_scan_kernel(uint32_t first, uint32_t count,
                                                                 uint32_t* need) {
  __shared__ uint32_t part[kScanThreads];
  const uint32_t per = (count + kScanThreads - 1) / kScanThreads;
  const uint32_t b = first + min(count, threadIdx.x * per), e = first + min(count, (threadIdx.x + 1) * per);
  uint32_t m = 0;
  for (uint32_t i = b; i < e; ++i) m = max(m, need[i]);
  part[threadIdx.x] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t run = 0;
    for (int t = 0; t < kScanThreads; ++t) { const uint32_t v = part[t]; part[t] = run; run = max(run, v); }
  }
  __syncthreads();
  m = part[threadIdx.x];                                  // maximum over the chunks before mine
  for (uint32_t i = b; i < e; ++i) { m = max(m, need[i]); need[i] = m; }
}

// ------------------------------------------------------------------------------- reset
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
    rs.load = 0; rs.min_fin = d_inf(); rs.occ = 0; rs.cur_req = kNone; rs.cur_pos = -1;
    rs.lru_tail = kNone;
    rep[i] = rs;
  }
  double* slot_d = reinterpret_cast<double*>(st + lay.slot_d_off);
  uint32_t* slot_u = reinterpret_cast<uint32_t*>(st + lay.slot_u_off);
  const uint32_t RS = R * S;
  for (uint32_t x = threadIdx.x; x < RS; x += blockDim.x) {
    slot_d[x] = 0.0;                    // free_at
    slot_d[RS + x] = d_inf();           // q0_fin
    slot_d[2 * (size_t)RS + x] = d_inf();   // q1_fin
    slot_u[x] = 0; slot_u[RS + x] = 0;  // q0_tok, q1_tok
    slot_u[2 * (size_t)RS + x] = kNone; // q2_idx
    slot_u[3 * (size_t)RS + x] = kNone; // tail
    slot_u[4 * (size_t)RS + x] = 0;     // qcnt
  }
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
  a.slots_in_smem = rs * 44 <= 44 * 1024 ? 1u : 0u;
  a.lists_in_smem = list_bytes <= 64 * 1024 ? 1u : 0u;
  return smem_plan(a.m.R, a.m.G, a.m.S, a.m.K, (uint32_t)sizeof(MaskT), a.slots_in_smem != 0,
                   a.lists_in_smem != 0).total;
}

template <typename MaskT>
cudaError_t launch_replay_t(ReplayArgs a, uint32_t n_cand, cudaStream_t st) {
  const size_t smem = replay_smem_bytes<MaskT>(a);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(replay_kernel<MaskT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  // several candidates share an SM (P is usually larger than the SM count): ask for the largest
  // shared-memory carve-out so that the per-CTA footprint, not the default split, decides
  {
    cudaError_t e = cudaFuncSetAttribute(replay_kernel<MaskT>,
                                         cudaFuncAttributePreferredSharedMemoryCarveout,
                                         (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
  }
  // which earlier requests can have finished by the arrival of each request (all candidates)
  {
    cudaError_t e = cudaMemsetAsync(a.need_svc + a.first, 0, (size_t)a.count * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    need_scatter_kernel<<<(a.count + 255) / 256, 256, 0, st>>>(a.tr.req, a.scale, a.m.tpot_ms,
                                                               a.first, a.count, a.need_svc, a.tq);
    need_scan_kernel<<<1, kScanThreads, 0, st>>>(a.first, a.count, a.need_svc);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  replay_kernel<MaskT><<<n_cand, kReplayThreads, smem, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

template <typename MaskT>
int replay_occupancy_t(ReplayArgs a, size_t* smem_out) {
  const size_t smem = replay_smem_bytes<MaskT>(a);
  *smem_out = smem;
  cudaFuncSetAttribute(replay_kernel<MaskT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  cudaFuncSetAttribute(replay_kernel<MaskT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                       (int)cudaSharedmemCarveoutMaxShared);
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, replay_kernel<MaskT>, (int)kReplayThreads,
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

cudaError_t launch_reset(unsigned char* masks, uint64_t mask_bytes_total, unsigned char* states,
                         const StateLayout& lay, const Model& m, uint32_t n_cand,
                         cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(masks, 0, mask_bytes_total, st);
  if (e != cudaSuccess) return e;
  reset_states_kernel<<<n_cand, 128, 0, st>>>(states, lay, m.R, m.S, n_cand);
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

cudaError_t launch_digest(const DigestArgs& a, uint32_t n_cand, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(a.digest, 0, (size_t)n_cand * a.m.R * 2 * sizeof(uint64_t), st);
  if (e != cudaSuccess) return e;
  const uint32_t chunks = 64;
  digest_kernel<<<dim3(n_cand, chunks), 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace gorgo

#ifdef GORGO_PROF
namespace gorgo {
int prof_read(unsigned long long* out, int clear) {
  cudaDeviceSynchronize();
  if (cudaMemcpyFromSymbol(out, g_prof, sizeof(g_prof)) != cudaSuccess) return -1;
  if (clear) {
    static unsigned long long z[256];
    cudaMemcpyToSymbol(g_prof, z, sizeof(z));
  }
  return 0;
}
}  // namespace gorgo
extern "C" int gorgo_prof_read(unsigned long long* out, int clear) { return gorgo::prof_read(out, clear); }
#endif

// TEST INFRASTRUCTURE ONLY -- plain, slow, single-threaded CPU statement of the routing
// simulator.  Nothing in the product path may link, import or call this file; it shares no
// code, header, table or helper with the CUDA library.  It exists so that tests (and the
// timed CPU baseline of the benchmark) have an independent definition to compare against.
//
// What it computes, per cost-model candidate, for each request of a Mooncake-style trace in
// trace order (paper Section 2.2, Eq. 1-3, and Section 2.3):
//   * the longest cached prefix (in 512-token blocks) of the request on every replica
//     (Section 1: prefix caching removes the prefill of earlier turns; Section 4 "prefix-cache"
//     baseline: proxy-side index of dispatched requests),
//   * the proxy-recorded queue signal: total input tokens of requests dispatched to a replica
//     that have no completion event yet (text below Eq. 1),
//   * the weighted score of Eq. 3 with explicit weights (w_net, w_prefill, w_queue) and the
//     argmin replica,
//   * an LRU block cache and a slot/queue service model per replica (the paper calls for
//     "a sufficiently accurate simulator of cache and continuous-batching dynamics",
//     Section 2.1, without giving one; the model here is this project's explicit statement),
//   * TTFT = network + queue wait + prefill of the uncached tokens (Eq. 1) and E2E latency,
//     reduced to their p95 (Section 4: the tuning objective is p95 TTFT).
//
// Pinned by tests/test_oracle_*.py: hand-worked traces, brute-force prefix matching, an
// independently written list-based LRU, Lindley's recursion, closed forms and invariants.
// Parity unpinned: the absolute TTFT/E2E values against the paper's tables (they need the
// paper's engines, model and trace).
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC gorgo_oracle.cpp -o libgorgo_oracle.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <set>
#include <unordered_map>
#include <utility>
#include <vector>

namespace {

// Recency key of a cached block: request index of its last touch and its position in that
// request.  Eviction order: smaller seq first; inside one request the DEEPEST block first, so
// a cache filled by prefix-sharing requests stays prefix-closed.
struct Key {
    uint64_t seq;
    uint32_t pos;
};
struct KeyEvictsBefore {
    bool operator()(const Key& a, const Key& b) const {
        if (a.seq != b.seq) return a.seq < b.seq;
        return a.pos > b.pos;
    }
};

struct Replica {
    std::unordered_map<uint64_t, Key> cache;              // block id -> recency key
    std::map<Key, uint64_t, KeyEvictsBefore> order;       // recency key -> block id
    std::vector<double> free_at;                          // per slot: time it becomes free
    std::vector<uint64_t> kv;                             // per slot: KV tokens of its newest request
    std::set<uint64_t> index;                             // the proxy's index: blocks ever dispatched here
    std::multiset<std::pair<double, uint64_t>> inflight;  // (finish time, input tokens)
    int64_t load = 0;                                     // sum of in-flight input tokens
};

uint64_t mix64(uint64_t z) {  // splitmix64 finaliser (Steele, Lea, Flood 2014)
    z ^= z >> 30;
    z *= 0xbf58476d1ce4e5b9ULL;
    z ^= z >> 27;
    z *= 0x94d049bb133111ebULL;
    z ^= z >> 31;
    return z;
}

struct Oracle {
    uint32_t R, G, S, B, K;
    uint64_t C;
    double prefill_ms, tpot_ms;
    std::vector<double> rtt;  // [G][R]
    uint64_t N;
    std::vector<double> ts;
    std::vector<uint32_t> in_tok, out_tok;
    std::vector<uint16_t> origin;
    std::vector<uint64_t> off, ids;
    std::vector<Replica> rep;
    uint64_t next = 0;        // next request to process
    uint64_t stats[4] = {0, 0, 0, 0};  // sum_i min(h_i+1,n), sum h*, sum n, sum evicted
    // Baseline policies of Section 4 inside the same simulator:
    //  * queue signal counted in requests instead of tokens ("least-request": the replica with
    //    the fewest in-flight requests from the proxy; in flight as for the token signal);
    //  * routes fixed in advance, one per request ("simple-session-affinity", "random": the
    //    choice does not depend on the simulator's state; the caller derives it).
    bool queue_in_requests = false;
    std::vector<uint8_t> forced_route;   // empty: route by the score
    // Heterogeneous replicas (the paper's Section 7 names them as a limitation of its uniform
    // fleet): per-replica prefill time per token and time per output token; empty = the uniform
    // constants.  The cost model does not see them (the proxy has no such signal).
    std::vector<double> rep_prefill_ms, rep_tpot_ms;
    // Continuous batching "bounded by max concurrency and KV budget" (Section 2.2), and the decode
    // slow-down of a fuller batch that makes concentrating traffic on one replica cost E2E latency
    // (Section 5, Appendix D).  Both are this project's statement, off by default:
    //  * decode_slowdown g >= 0: a request's time per output token is tpot * (1 + g*(b-1)), b = the
    //    replica's busy slots at its first-token time, itself included;
    //  * kv_budget > 0: a request needing in+out tokens of KV starts only once the newest requests of
    //    the other busy slots hold at most kv_budget - need tokens (it runs alone whatever its size).
    double decode_slowdown = 0.0;
    uint64_t kv_budget = 0;
    // Time-varying network (paper Section 2.2: the proxy's RTT signal is an exponentially weighted
    // moving average of a probe sent every 30 s).  rtt_raw[e][g][i] is the probe result of epoch e,
    // which is also the delay a request dispatched in that epoch experiences; rtt_ewma[e][g][i] is
    // what the proxy believes during epoch e and puts into the score.  Empty = the static matrix.
    std::vector<double> rtt_raw, rtt_ewma;
    uint32_t n_epochs = 0;
    double epoch_ms = 0.0;
    // Proxy index that drifts from the replica's cache (paper Section 7: the proxy's prefix index is
    // built from the requests it dispatched and does not observe what the replica evicts).  When
    // on, the score of Eq. 3 takes the prefix hit from the index -- every block ever dispatched to
    // the replica, never forgotten -- while prefill time, the reported hit and the cache itself
    // follow the replica's real LRU cache.
    bool proxy_index = false;
};

// Epoch of (scaled) time t: the largest k in [0, n_epochs-1] with k * epoch_ms <= t.
uint32_t epoch_of(const Oracle* o, double t) {
    uint32_t k = 0;
    while (k + 1 < o->n_epochs && (double)(k + 1) * o->epoch_ms <= t) ++k;
    return k;
}

}  // namespace

extern "C" {

struct gorgo_oracle_config {
    uint32_t n_replicas, n_regions, slots_per_replica, block_tokens;
    uint64_t cache_blocks;
    uint32_t n_params;
    uint32_t _pad;
    double prefill_ms_per_token, tpot_ms;
};

// Copies everything; returns NULL on a malformed configuration.
void* gorgo_oracle_create(const gorgo_oracle_config* cfg, const double* rtt_ms,
                          uint64_t n_requests, const double* ts_ms, const uint32_t* input_tokens,
                          const uint32_t* output_tokens, const uint16_t* origin,
                          const uint64_t* hash_off, const uint64_t* hash_ids) {
    if (!cfg || !rtt_ms || cfg->n_replicas == 0 || cfg->n_regions == 0 ||
        cfg->slots_per_replica == 0 || cfg->block_tokens == 0)
        return nullptr;
    if (cfg->n_params != 3 && cfg->n_params != 3 + cfg->n_replicas) return nullptr;
    Oracle* o = new Oracle();
    o->R = cfg->n_replicas; o->G = cfg->n_regions; o->S = cfg->slots_per_replica;
    o->B = cfg->block_tokens; o->K = cfg->n_params; o->C = cfg->cache_blocks;
    o->prefill_ms = cfg->prefill_ms_per_token; o->tpot_ms = cfg->tpot_ms;
    o->rtt.assign(rtt_ms, rtt_ms + (size_t)o->G * o->R);
    o->N = n_requests;
    o->ts.assign(ts_ms, ts_ms + n_requests);
    o->in_tok.assign(input_tokens, input_tokens + n_requests);
    o->out_tok.assign(output_tokens, output_tokens + n_requests);
    if (origin) o->origin.assign(origin, origin + n_requests);
    else o->origin.assign(n_requests, 0);
    o->off.assign(hash_off, hash_off + n_requests + 1);
    o->ids.assign(hash_ids, hash_ids + hash_off[n_requests]);
    o->rep.resize(o->R);
    for (auto& rp : o->rep) { rp.free_at.assign(o->S, 0.0); rp.kv.assign(o->S, 0); }
    return o;
}

void gorgo_oracle_destroy(void* h) { delete static_cast<Oracle*>(h); }

// Back to the empty state (no cached blocks, all slots free at time 0, nothing in flight).
void gorgo_oracle_reset(void* h) {
    Oracle* o = static_cast<Oracle*>(h);
    for (auto& rp : o->rep) {
        rp.cache.clear(); rp.order.clear(); rp.inflight.clear(); rp.index.clear();
        rp.free_at.assign(o->S, 0.0); rp.kv.assign(o->S, 0); rp.load = 0;
    }
    o->next = 0;
    std::memset(o->stats, 0, sizeof(o->stats));
}

// Routes the next `count` requests with cost-model parameters w[0..K) and timestamp scale
// `scale`, committing cache and queue state.  All outputs are optional (NULL) and indexed from
// the first request of this call.  Returns the number of requests processed.
//   route[j], hit[j]        chosen replica and its prefix-hit length in blocks
//   ttft[j], e2e[j]         simulated latencies in ms
//   hit_all[j*R+i]          prefix-hit length on every replica (before the commit)
//   load_all[j*R+i]         in-flight input tokens on every replica as seen by the score
//   cost_all[j*R+i]         the score of Eq. 3
//   evicted[j]              blocks evicted from the chosen replica by this request
//   occ_after[j]            occupancy of the chosen replica after the commit
uint64_t gorgo_oracle_run(void* h, const double* w, double scale, uint64_t count,
                          uint8_t* route, uint16_t* hit, double* ttft, double* e2e,
                          uint16_t* hit_all, int64_t* load_all, double* cost_all,
                          uint32_t* evicted, uint64_t* occ_after) {
    Oracle* o = static_cast<Oracle*>(h);
    const uint32_t R = o->R;
    std::vector<uint64_t> hits(R), unc(R);
    std::vector<double> cost(R);
    uint64_t done = 0;
    for (; done < count && o->next < o->N; ++done, ++o->next) {
        const uint64_t r = o->next;
        const double t = scale * o->ts[r];                 // scaled arrival time at the proxy
        const uint32_t g = o->origin[r];
        const uint64_t n = o->off[r + 1] - o->off[r];
        const uint64_t* id = o->ids.data() + o->off[r];
        const uint64_t in = o->in_tok[r];
        // the proxy's RTT signal and the delay of the network at this time
        const double* rtt_signal = o->rtt.data() + (size_t)g * R;
        const double* rtt_delay = rtt_signal;
        if (o->n_epochs > 0) {
            const size_t e = epoch_of(o, t);
            rtt_signal = o->rtt_ewma.data() + (e * o->G + g) * R;
            rtt_delay = o->rtt_raw.data() + (e * o->G + g) * R;
        }

        for (uint32_t i = 0; i < R; ++i) {
            Replica& rp = o->rep[i];
            // completion events seen by the proxy: finish <= t is no longer in flight
            while (!rp.inflight.empty() && rp.inflight.begin()->first <= t) {
                rp.load -= (int64_t)rp.inflight.begin()->second;
                rp.inflight.erase(rp.inflight.begin());
            }
            // longest cached prefix, stop at the first missing block
            uint64_t hh = 0;
            while (hh < n && rp.cache.count(id[hh])) ++hh;
            hits[i] = hh;
            unc[i] = in - std::min<uint64_t>(hh * o->B, in);
            uint64_t unc_score = unc[i];                   // what the proxy believes is uncached
            if (o->proxy_index) {
                uint64_t hb = 0;
                while (hb < n && rp.index.count(id[hb])) ++hb;
                unc_score = in - std::min<uint64_t>(hb * o->B, in);
            }
            double q = o->queue_in_requests ? (double)rp.inflight.size() : (double)rp.load;
            if (o->K != 3) q = q * w[3 + i];               // per-replica queue-load normaliser
            // Eq. 3 with explicit weights: three products, two sums, in this order
            const double a = w[0] * rtt_signal[i];
            const double b = w[1] * (double)unc_score;
            const double c = w[2] * q;
            cost[i] = (a + b) + c;
            if (hit_all) hit_all[done * R + i] = (uint16_t)hh;
            if (load_all) load_all[done * R + i] = rp.load;
            if (cost_all) cost_all[done * R + i] = cost[i];
            o->stats[0] += std::min<uint64_t>(hh + 1, n);
        }
        uint32_t best = 0;                                 // lowest index wins ties
        for (uint32_t i = 1; i < R; ++i)
            if (cost[i] < cost[best]) best = i;
        if (!o->forced_route.empty()) best = o->forced_route[r];

        // ---- cache commit on the chosen replica (set semantics) ----
        Replica& rp = o->rep[best];
        std::vector<char> present(n, 0);
        uint64_t missing = 0;
        for (uint64_t k = 0; k < n; ++k) {
            auto it = rp.cache.find(id[k]);
            if (it != rp.cache.end()) {
                present[k] = 1;
                rp.order.erase(it->second);
                it->second = Key{r, (uint32_t)k};
                rp.order.emplace(it->second, id[k]);
            } else {
                ++missing;
            }
        }
        uint64_t occ = rp.cache.size();
        uint64_t E = (occ + missing > o->C) ? (occ + missing - o->C) : 0;
        uint32_t ev = 0;
        while (E > 0) {
            auto victim = rp.order.begin();                // smallest key; never of this request
            if (victim == rp.order.end() || victim->first.seq == r) break;
            rp.cache.erase(victim->second);
            rp.order.erase(victim);
            --E; ++ev;
        }
        for (uint64_t k = 0; k < n; ++k) {
            if (!present[k]) {
                Key key{r, (uint32_t)k};
                rp.cache.emplace(id[k], key);
                rp.order.emplace(key, id[k]);
            }
        }

        if (o->proxy_index) rp.index.insert(id, id + n);   // the proxy learns what it dispatched

        // ---- service commit on the chosen replica ----
        const double arrive = t + rtt_delay[best];
        uint32_t slot = 0;
        for (uint32_t s = 1; s < o->S; ++s)
            if (rp.free_at[s] < rp.free_at[slot]) slot = s;
        double start = std::max(arrive, rp.free_at[slot]);
        const uint32_t out = o->out_tok[r];
        const uint64_t need = in + out;                    // KV tokens the request holds while it runs
        if (o->kv_budget > 0) {
            // admission under the KV budget: wait for other slots to finish until the request fits
            for (;;) {
                uint64_t usage = 0;
                double next_free = 0.0;
                bool any_busy = false;
                for (uint32_t s = 0; s < o->S; ++s) {
                    if (s == slot || !(rp.free_at[s] > start)) continue;
                    usage += rp.kv[s];
                    if (!any_busy || rp.free_at[s] < next_free) next_free = rp.free_at[s];
                    any_busy = true;
                }
                if (!any_busy || usage + need <= o->kv_budget) break;
                start = next_free;
            }
        }
        const double prefill =
            (o->rep_prefill_ms.empty() ? o->prefill_ms : o->rep_prefill_ms[best]) * (double)unc[best];
        const double first = start + prefill;
        double tpot = o->rep_tpot_ms.empty() ? o->tpot_ms : o->rep_tpot_ms[best];
        if (o->decode_slowdown > 0.0) {
            uint32_t busy = 1;                             // slots busy at the first token, this one included
            for (uint32_t s = 0; s < o->S; ++s)
                if (s != slot && rp.free_at[s] > first) ++busy;
            const double g = 1.0 + o->decode_slowdown * (double)(busy - 1);
            tpot = tpot * g;
        }
        const double decode = tpot * (double)(out > 0 ? out - 1 : 0);
        const double finish = first + decode;
        rp.free_at[slot] = finish;
        rp.kv[slot] = need;
        rp.inflight.emplace(finish, in);
        rp.load += (int64_t)in;

        if (route) route[done] = (uint8_t)best;
        if (hit) hit[done] = (uint16_t)hits[best];
        if (ttft) ttft[done] = first - t;
        if (e2e) e2e[done] = finish - t;
        if (evicted) evicted[done] = ev;
        if (occ_after) occ_after[done] = rp.cache.size();
        o->stats[1] += hits[best];
        o->stats[2] += n;
        o->stats[3] += ev;
    }
    return done;
}

// Baseline-policy switches (see the Oracle struct).  `forced_route` holds one replica index per
// request of the trace, or is NULL to route by the score again.  Returns 0, or -1 if an index is
// out of range.
int gorgo_oracle_set_policy(void* h, uint32_t queue_in_requests, const uint8_t* forced_route) {
    Oracle* o = static_cast<Oracle*>(h);
    if (forced_route)
        for (uint64_t r = 0; r < o->N; ++r)
            if (forced_route[r] >= o->R) return -1;
    o->queue_in_requests = queue_in_requests != 0;
    if (forced_route) o->forced_route.assign(forced_route, forced_route + o->N);
    else o->forced_route.clear();
    return 0;
}

// Per-replica service speeds (R values each, NULL = the uniform constant).  Returns 0, or -1 for a
// negative or non-finite value.
int gorgo_oracle_set_replica_speeds(void* h, const double* prefill_ms_per_token,
                                    const double* tpot_ms) {
    Oracle* o = static_cast<Oracle*>(h);
    for (uint32_t i = 0; i < o->R; ++i) {
        if (prefill_ms_per_token && !(prefill_ms_per_token[i] >= 0.0 && std::isfinite(prefill_ms_per_token[i]))) return -1;
        if (tpot_ms && !(tpot_ms[i] >= 0.0 && std::isfinite(tpot_ms[i]))) return -1;
    }
    if (prefill_ms_per_token) o->rep_prefill_ms.assign(prefill_ms_per_token, prefill_ms_per_token + o->R);
    else o->rep_prefill_ms.clear();
    if (tpot_ms) o->rep_tpot_ms.assign(tpot_ms, tpot_ms + o->R);
    else o->rep_tpot_ms.clear();
    return 0;
}

// Decode slow-down per additional busy slot (>= 0, finite) and KV budget in tokens per replica
// (0 = unlimited).  Returns 0, or -1 for a bad value.
int gorgo_oracle_set_service_model(void* h, double decode_slowdown, uint64_t kv_budget_tokens) {
    Oracle* o = static_cast<Oracle*>(h);
    if (!(decode_slowdown >= 0.0 && std::isfinite(decode_slowdown))) return -1;
    o->decode_slowdown = decode_slowdown;
    o->kv_budget = kv_budget_tokens;
    return 0;
}

// Proxy index separate from the replica's cache (see the Oracle struct); takes effect from the
// empty state.
void gorgo_oracle_set_proxy_index(void* h, uint32_t on) { static_cast<Oracle*>(h)->proxy_index = on != 0; }

// Probe results per epoch, samples[e][g][i] >= 0, one epoch every epoch_ms > 0 of (scaled) time,
// smoothing factor 0 < alpha <= 1.  The proxy's signal is ewma_0 = s_0,
// ewma_e = ewma_{e-1} + alpha * (s_e - ewma_{e-1}) (three rounded operations).  n_epochs = 0
// restores the static matrix.  Returns 0, or -1 for a bad argument.
int gorgo_oracle_set_rtt_series(void* h, uint32_t n_epochs, double epoch_ms, double alpha,
                                const double* samples) {
    Oracle* o = static_cast<Oracle*>(h);
    if (n_epochs == 0) { o->n_epochs = 0; o->rtt_raw.clear(); o->rtt_ewma.clear(); return 0; }
    if (!samples || !(epoch_ms > 0.0) || !std::isfinite(epoch_ms) || !(alpha > 0.0 && alpha <= 1.0)) return -1;
    const size_t gr = (size_t)o->G * o->R;
    for (size_t x = 0; x < n_epochs * gr; ++x)
        if (!(samples[x] >= 0.0 && std::isfinite(samples[x]))) return -1;
    o->rtt_raw.assign(samples, samples + n_epochs * gr);
    o->rtt_ewma.assign(samples, samples + n_epochs * gr);
    for (uint32_t e = 1; e < n_epochs; ++e)
        for (size_t x = 0; x < gr; ++x) {
            const double prev = o->rtt_ewma[(e - 1) * gr + x];
            const double diff = samples[e * gr + x] - prev;
            const double step = alpha * diff;
            o->rtt_ewma[e * gr + x] = prev + step;
        }
    o->n_epochs = n_epochs;
    o->epoch_ms = epoch_ms;
    return 0;
}

// Nearest-rank percentile: the k-th smallest with k = ceil(0.95 n) in integers.
double gorgo_oracle_p95(const double* v, uint64_t n) {
    if (n == 0) return 0.0;
    std::vector<double> s(v, v + n);
    std::sort(s.begin(), s.end());
    const uint64_t k = (95 * n + 99) / 100;
    return s[k - 1];
}

// out[2*i] = occupancy of replica i, out[2*i+1] = order-independent sum (mod 2^64) over its
// cached blocks of mix64(id ^ mix64(seq*65536 + pos)).
void gorgo_oracle_digest(void* h, uint64_t* out) {
    Oracle* o = static_cast<Oracle*>(h);
    for (uint32_t i = 0; i < o->R; ++i) {
        uint64_t sum = 0;
        for (const auto& kv : o->rep[i].cache)
            sum += mix64(kv.first ^ mix64(kv.second.seq * 65536ULL + kv.second.pos));
        out[2 * i] = o->rep[i].cache.size();
        out[2 * i + 1] = sum;
    }
}

// Cached blocks of one replica in eviction order (first = next victim).  Returns the
// occupancy; writes at most `cap` entries.
uint64_t gorgo_oracle_dump(void* h, uint32_t replica, uint64_t cap, uint64_t* ids,
                           uint64_t* seq, uint32_t* pos) {
    Oracle* o = static_cast<Oracle*>(h);
    uint64_t j = 0;
    for (const auto& kv : o->rep[replica].order) {
        if (j < cap) {
            if (ids) ids[j] = kv.second;
            if (seq) seq[j] = kv.first.seq;
            if (pos) pos[j] = kv.first.pos;
        }
        ++j;
    }
    return j;
}

// loads[i] = in-flight input tokens, inflight[i] = number of in-flight requests (as of the
// last processed request), free_at[i*S+s] = slot release times.
void gorgo_oracle_queues(void* h, int64_t* loads, uint64_t* inflight, double* free_at) {
    Oracle* o = static_cast<Oracle*>(h);
    for (uint32_t i = 0; i < o->R; ++i) {
        if (loads) loads[i] = o->rep[i].load;
        if (inflight) inflight[i] = o->rep[i].inflight.size();
        if (free_at)
            for (uint32_t s = 0; s < o->S; ++s) free_at[(size_t)i * o->S + s] = o->rep[i].free_at[s];
    }
}

void gorgo_oracle_stats(void* h, uint64_t* out4) {
    Oracle* o = static_cast<Oracle*>(h);
    std::memcpy(out4, o->stats, sizeof(o->stats));
}

uint64_t gorgo_oracle_position(void* h) { return static_cast<Oracle*>(h)->next; }

}  // extern "C"

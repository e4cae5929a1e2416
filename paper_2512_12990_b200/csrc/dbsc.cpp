// Host-side Dynamic Bit-Sliced Caching bookkeeping (Section 4.1 of the paper).  Plain C++; no CUDA.
//
// Two intrusive orderings over cached slices: MSB slices in LRU order, LSB slices in insertion
// order.  Eviction always drains the LSB queue (oldest first) before touching the MSB list (least
// recently used first).  Keys are (layer, expert); one cache serves all layers.
//
// Predictive Cache Warmup (Section 4.3): while a prompt is prefilled layer by layer the cache takes the
// slices of every expert the layer used and, whenever it overflows, drops the LSB slice with the lowest
// gating score, or - once no LSB slice is left - the MSB slice with the lowest prefill access frequency.
// At the end of prefill both orderings are rebuilt from the accumulated statistics.
#include <algorithm>
#include <cstdint>
#include <list>
#include <new>
#include <tuple>
#include <unordered_map>
#include <vector>

#include "slicemoe.h"

namespace {

inline uint64_t make_key(int layer, int expert) {
  return (static_cast<uint64_t>(static_cast<uint32_t>(layer)) << 32) | static_cast<uint32_t>(expert);
}

struct Queue {
  std::list<uint64_t> order;  // front = next victim
  std::unordered_map<uint64_t, std::list<uint64_t>::iterator> where;

  bool has(uint64_t k) const { return where.find(k) != where.end(); }
  void push_back(uint64_t k) {
    order.push_back(k);
    where[k] = std::prev(order.end());
  }
  void touch(uint64_t k) {  // move to the most-recently-used end
    auto it = where.find(k);
    order.splice(order.end(), order, it->second);
  }
  void erase(uint64_t k) {
    auto it = where.find(k);
    order.erase(it->second);
    where.erase(it);
  }
  // Removes the first entry that is not `protect` (and names it); false if there is none.
  bool evict_one(uint64_t protect, uint64_t* victim) {
    for (auto it = order.begin(); it != order.end(); ++it) {
      if (*it != protect) {
        *victim = *it;
        where.erase(*it);
        order.erase(it);
        return true;
      }
    }
    return false;
  }
};

}  // namespace

struct slicemoe_dbsc {
  int64_t capacity, msb_bytes, lsb_bytes, used;
  double miss_budget;
  int warmup_steps;
  Queue msb, lsb;
  int64_t requests, msb_hit, msb_miss, lsb_hit, lsb_miss, lsb_skipped, bytes_fetched, high_exec, low_exec,
      win_fetched, win_full;
  struct Hotness { int64_t freq; double score; };  // prompt tokens routed to the expert; their mean gating score
  std::unordered_map<uint64_t, Hotness> hot;       // statistics of the prefill in progress
  // For a caller that keeps the slices themselves (slicemoe_tier): what request() evicted, until it is drained.
  bool log_evictions = false;
  std::vector<std::pair<uint64_t, int>> evicted;   // (key, 1 = LSB slice)

  // Eviction keys of Section 4.3; a slice without statistics (left from before the prompt) goes first.
  std::tuple<double, int64_t, uint64_t> lsb_rank(uint64_t k) const {
    auto it = hot.find(k);
    return it == hot.end() ? std::make_tuple(-1.0, int64_t(-1), k) : std::make_tuple(it->second.score, it->second.freq, k);
  }
  std::tuple<int64_t, double, uint64_t> msb_rank(uint64_t k) const {
    auto it = hot.find(k);
    return it == hot.end() ? std::make_tuple(int64_t(-1), -1.0, k) : std::make_tuple(it->second.freq, it->second.score, k);
  }

  void prefill_layer(int layer, const std::vector<int64_t>& freq, const std::vector<double>& sum, double tau) {
    for (size_t e = 0; e < freq.size(); ++e) {
      if (freq[e] <= 0) continue;
      const uint64_t key = make_key(layer, static_cast<int>(e));
      const double score = sum[e] / static_cast<double>(freq[e]);
      hot[key] = Hotness{freq[e], score};
      if (!msb.has(key)) {
        msb.push_back(key);
        used += msb_bytes;
      }
      if (score >= tau && !lsb.has(key)) {
        lsb.push_back(key);
        used += lsb_bytes;
      }
    }
    if (used <= capacity) return;
    // victims in order: slices from before the prompt (LSB, then MSB), then the prompt's LSB slices by score,
    // then its MSB slices by frequency
    std::vector<uint64_t> lv(lsb.order.begin(), lsb.order.end()), mv(msb.order.begin(), msb.order.end());
    std::sort(lv.begin(), lv.end(), [&](uint64_t a, uint64_t b) { return lsb_rank(a) < lsb_rank(b); });
    std::sort(mv.begin(), mv.end(), [&](uint64_t a, uint64_t b) { return msb_rank(a) < msb_rank(b); });
    size_t li = 0, mi = 0;
    for (; li < lv.size() && !hot.count(lv[li]) && used > capacity; ++li) {
      lsb.erase(lv[li]);
      used -= lsb_bytes;
    }
    for (; mi < mv.size() && !hot.count(mv[mi]) && used > capacity; ++mi) {
      msb.erase(mv[mi]);
      used -= msb_bytes;
    }
    for (; li < lv.size() && used > capacity; ++li) {
      lsb.erase(lv[li]);
      used -= lsb_bytes;
    }
    for (; mi < mv.size() && used > capacity; ++mi) {
      msb.erase(mv[mi]);
      used -= msb_bytes;
    }
  }

  void prefill_end() {
    std::vector<uint64_t> lv(lsb.order.begin(), lsb.order.end()), mv(msb.order.begin(), msb.order.end());
    std::sort(lv.begin(), lv.end(), [&](uint64_t a, uint64_t b) { return lsb_rank(a) < lsb_rank(b); });
    std::sort(mv.begin(), mv.end(), [&](uint64_t a, uint64_t b) { return msb_rank(a) < msb_rank(b); });
    Queue nl, nm;
    for (uint64_t k : lv) nl.push_back(k);
    for (uint64_t k : mv) nm.push_back(k);
    lsb = std::move(nl);
    msb = std::move(nm);
    hot.clear();
  }

  bool make_room(int64_t need, uint64_t protect) {
    if (need > capacity) return false;
    while (capacity - used < need) {
      uint64_t victim = 0;
      if (lsb.evict_one(protect, &victim)) {
        used -= lsb_bytes;
        if (log_evictions) evicted.emplace_back(victim, 1);
      } else if (msb.evict_one(protect, &victim)) {
        used -= msb_bytes;
        if (log_evictions) evicted.emplace_back(victim, 0);
      } else {
        return false;
      }
    }
    return true;
  }

  bool over_budget(int step) const {
    if (miss_budget < 0.0 || step < warmup_steps || win_full <= 0) return false;
    return static_cast<double>(win_fetched) / static_cast<double>(win_full) > miss_budget;
  }

  int request(int step, int layer, int expert, bool need_lsb, int* msb_hit_out, int* lsb_hit_out,
              int64_t* fetched_out) {
    const uint64_t key = make_key(layer, expert);
    ++requests;
    int64_t fetched = 0;
    int mh, lh = -1, prec = 0;
    if (msb.has(key)) {
      msb.touch(key);
      mh = 1;
      ++msb_hit;
    } else {
      mh = 0;
      ++msb_miss;
      fetched += msb_bytes;
      if (make_room(msb_bytes, key)) {
        msb.push_back(key);
        used += msb_bytes;
      }
    }
    if (need_lsb) {
      if (lsb.has(key)) {
        lh = 1;
        ++lsb_hit;
        prec = 1;
      } else {
        lh = 0;
        if (over_budget(step)) {
          ++lsb_skipped;
        } else {
          ++lsb_miss;
          fetched += lsb_bytes;
          prec = 1;
          if (make_room(lsb_bytes, key)) {
            lsb.push_back(key);
            used += lsb_bytes;
          }
        }
      }
    }
    bytes_fetched += fetched;
    if (prec) ++high_exec; else ++low_exec;
    if (step >= warmup_steps) {
      win_fetched += fetched;
      win_full += msb_bytes + lsb_bytes;
    }
    if (msb_hit_out) *msb_hit_out = mh;
    if (lsb_hit_out) *lsb_hit_out = lh;
    if (fetched_out) *fetched_out = fetched;
    return prec;
  }
};

extern "C" slicemoe_dbsc* slicemoe_dbsc_create(int64_t capacity_bytes, int64_t msb_bytes, int64_t lsb_bytes,
                                               double miss_budget, int warmup_steps) {
  if (capacity_bytes < 0 || msb_bytes <= 0 || lsb_bytes <= 0 || warmup_steps < 0) return nullptr;
  slicemoe_dbsc* c = new (std::nothrow) slicemoe_dbsc();
  if (!c) return nullptr;
  c->capacity = capacity_bytes;
  c->msb_bytes = msb_bytes;
  c->lsb_bytes = lsb_bytes;
  c->used = 0;
  c->miss_budget = miss_budget;
  c->warmup_steps = warmup_steps;
  c->requests = c->msb_hit = c->msb_miss = c->lsb_hit = c->lsb_miss = c->lsb_skipped = 0;
  c->bytes_fetched = c->high_exec = c->low_exec = c->win_fetched = c->win_full = 0;
  return c;
}

extern "C" void slicemoe_dbsc_destroy(slicemoe_dbsc* c) { delete c; }

extern "C" int slicemoe_dbsc_request(slicemoe_dbsc* c, int step, int layer, int expert, int need_lsb,
                                     int* msb_hit, int* lsb_hit, int64_t* fetched_bytes) {
  if (!c || layer < 0 || expert < 0 || step < 0) return SLICEMOE_E_INVALID_ARG;
  try {
    return c->request(step, layer, expert, need_lsb != 0, msb_hit, lsb_hit, fetched_bytes);
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
}

extern "C" int slicemoe_dbsc_assign(slicemoe_dbsc* c, int step, int layer, const int32_t* ids,
                                    const uint8_t* prec_req, int n, uint8_t* prec_out) {
  if (!c || !ids || !prec_req || !prec_out || n < 0 || layer < 0 || step < 0) return SLICEMOE_E_INVALID_ARG;
  for (int i = 0; i < n; ++i)
    if (ids[i] < 0) return SLICEMOE_E_INVALID_ARG;
  try {
    for (int i = 0; i < n; ++i)
      prec_out[i] = static_cast<uint8_t>(c->request(step, layer, ids[i], prec_req[i] != 0, nullptr, nullptr, nullptr));
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
  return SLICEMOE_OK;
}

extern "C" int slicemoe_dbsc_stats(const slicemoe_dbsc* c, int64_t* out) {
  if (!c || !out) return SLICEMOE_E_INVALID_ARG;
  const int64_t v[SLICEMOE_DBSC_NSTATS] = {c->requests,   c->msb_hit,       c->msb_miss,  c->lsb_hit,
                                           c->lsb_miss,   c->lsb_skipped,   c->bytes_fetched, c->high_exec,
                                           c->low_exec,   c->win_fetched,   c->win_full,  c->used};
  for (int i = 0; i < SLICEMOE_DBSC_NSTATS; ++i) out[i] = v[i];
  return SLICEMOE_OK;
}

extern "C" int slicemoe_dbsc_contains(const slicemoe_dbsc* c, int layer, int expert, int* has_msb, int* has_lsb) {
  if (!c || layer < 0 || expert < 0) return SLICEMOE_E_INVALID_ARG;
  const uint64_t key = make_key(layer, expert);
  if (has_msb) *has_msb = c->msb.has(key) ? 1 : 0;
  if (has_lsb) *has_lsb = c->lsb.has(key) ? 1 : 0;
  return SLICEMOE_OK;
}

extern "C" int slicemoe_dbsc_prefill_layer(slicemoe_dbsc* c, int layer, const int32_t* ids, const float* scores,
                                           int64_t n_pairs, int n_experts, double tau) {
  if (!c || !ids || !scores || layer < 0 || n_pairs < 0 || n_experts <= 0) return SLICEMOE_E_INVALID_ARG;
  for (int64_t i = 0; i < n_pairs; ++i)
    if (ids[i] < 0 || ids[i] >= n_experts) return SLICEMOE_E_INVALID_ARG;
  try {
    std::vector<int64_t> freq(n_experts, 0);
    std::vector<double> sum(n_experts, 0.0);
    for (int64_t i = 0; i < n_pairs; ++i) {  // in list order: the sums are reproducible
      ++freq[ids[i]];
      sum[ids[i]] += static_cast<double>(scores[i]);
    }
    c->prefill_layer(layer, freq, sum, tau);
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
  return SLICEMOE_OK;
}

extern "C" int slicemoe_dbsc_prefill_end(slicemoe_dbsc* c) {
  if (!c) return SLICEMOE_E_INVALID_ARG;
  try {
    c->prefill_end();
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
  return SLICEMOE_OK;
}

extern "C" int slicemoe_dbsc_log_evictions(slicemoe_dbsc* c, int on) {
  if (!c) return SLICEMOE_E_INVALID_ARG;
  c->log_evictions = on != 0;
  if (!on) c->evicted.clear();
  return SLICEMOE_OK;
}

extern "C" int slicemoe_dbsc_drain_evicted(slicemoe_dbsc* c, int32_t* layers, int32_t* experts, uint8_t* is_lsb, int max) {
  if (!c || !layers || !experts || !is_lsb || max < 0) return SLICEMOE_E_INVALID_ARG;
  const int n = static_cast<int>(std::min<size_t>(c->evicted.size(), static_cast<size_t>(max)));
  for (int i = 0; i < n; ++i) {
    layers[i] = static_cast<int32_t>(c->evicted[i].first >> 32);
    experts[i] = static_cast<int32_t>(c->evicted[i].first & 0xffffffffu);
    is_lsb[i] = static_cast<uint8_t>(c->evicted[i].second);
  }
  c->evicted.erase(c->evicted.begin(), c->evicted.begin() + n);
  return n;
}

// ---- cache-aware routing baselines (Section 2.1; Section 6.1 "Baseline MoE Acceleration") -------------------
extern "C" int slicemoe_dbsc_bias(const slicemoe_dbsc* c, int layer, int n_experts, float delta, float* bias_out) {
  if (!c || !bias_out || layer < 0 || n_experts <= 0) return SLICEMOE_E_INVALID_ARG;
  for (int e = 0; e < n_experts; ++e) bias_out[e] = c->msb.has(make_key(layer, e)) ? delta : 0.0f;
  return SLICEMOE_OK;
}

extern "C" int slicemoe_cumsum_select(const float* probs, const uint8_t* cached, int n_experts, int k, double p,
                                      int32_t* ids_out) {
  if (!probs || !cached || !ids_out || n_experts <= 0 || k < 1 || k > n_experts) return SLICEMOE_E_INVALID_ARG;
  try {
    std::vector<int> order(n_experts);
    for (int e = 0; e < n_experts; ++e) order[e] = e;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return probs[a] > probs[b]; });
    // the shortest prefix that holds k experts and a probability mass of at least p (summed in double)
    int n = 0;
    double acc = 0.0;
    while (n < n_experts && (n < k || acc < p)) acc += static_cast<double>(probs[order[n++]]);
    int out = 0;
    for (int pass = 0; pass < 2 && out < k; ++pass)  // cached candidates first, each class in ranking order
      for (int i = 0; i < n && out < k; ++i)
        if ((cached[order[i]] != 0) == (pass == 0)) ids_out[out++] = order[i];
  } catch (...) {
    return SLICEMOE_E_NOMEM;
  }
  return SLICEMOE_OK;
}

// ---- the hardware cost model (Section 5) -------------------------------------------------------------------
extern "C" void slicemoe_cost_paper_hw(slicemoe_cost_hw* hw) {
  if (!hw) return;
  hw->dram_pj_per_bit = 1.5;
  hw->flash_pj_per_bit = 103.0;
  hw->dram_gbps = 104.0;
  hw->flash_gbps = 10.0;
  hw->tops = 16.4;
  hw->tops_per_watt = 3.18;
}

extern "C" int slicemoe_cost_step(const slicemoe_cost_hw* hw, int64_t flash_bytes, int64_t dram_bytes, int64_t macs,
                                  double* energy_joule, double* latency_s) {
  if (!hw || flash_bytes < 0 || dram_bytes < 0 || macs < 0) return SLICEMOE_E_INVALID_ARG;
  if (!(hw->dram_gbps > 0.0) || !(hw->flash_gbps > 0.0) || !(hw->tops > 0.0) || !(hw->tops_per_watt > 0.0))
    return SLICEMOE_E_INVALID_ARG;
  const double flash_bits = 8.0 * static_cast<double>(flash_bytes), dram_bits = 8.0 * static_cast<double>(dram_bytes);
  const double ops = 2.0 * static_cast<double>(macs);
  if (energy_joule)
    *energy_joule = flash_bits * hw->flash_pj_per_bit * 1e-12 + (flash_bits + dram_bits) * hw->dram_pj_per_bit * 1e-12 +
                    ops / (hw->tops_per_watt * 1e12);
  if (latency_s) {
    const double t_dram = dram_bits / (hw->dram_gbps * 1e9), t_compute = ops / (hw->tops * 1e12);
    *latency_s = flash_bits / (hw->flash_gbps * 1e9) + (t_dram > t_compute ? t_dram : t_compute);
  }
  return SLICEMOE_OK;
}

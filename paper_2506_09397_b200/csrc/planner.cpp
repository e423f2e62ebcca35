#include "planner.h"

#include <algorithm>
#include <cmath>
#include <queue>
#include <unordered_set>

#include "../../include/sled.h"

namespace sled {

Planner::Planner(int policy, int32_t batch_size, int32_t max_batch, int32_t max_step_tokens)
    : policy_(policy), batch_size_(batch_size), max_batch_(max_batch), max_step_tokens_(max_step_tokens) {
  valid_ = (policy == kBatchStatic || policy == kBatchContinuous) && max_batch > 0 && max_step_tokens > 0 &&
           (policy == kBatchContinuous || (batch_size > 0 && batch_size <= max_batch));
}

int Planner::push(uint64_t ticket, uint64_t ctx, int32_t k) {
  if (k < 0 || k + 1 > max_step_tokens_) return SLED_ERR_K_RANGE;   // could never be scheduled
  q_.push_back({ticket, ctx, k});
  return SLED_OK;
}

std::vector<uint64_t> Planner::next_batch(bool flush) {
  const int32_t limit = policy_ == kBatchStatic ? batch_size_ : max_batch_;
  // which queue entries the batch would take
  std::vector<size_t> take;
  std::unordered_set<uint64_t> seen;
  int64_t tokens = 0;
  bool step_full = false;                                   // the step's token capacity ended the scan
  for (size_t i = 0; i < q_.size() && static_cast<int32_t>(take.size()) < limit; ++i) {
    const QueuedRequest& r = q_[i];
    if (seen.count(r.ctx)) continue;                        // same context again: next step
    if (tokens + r.k + 1 > max_step_tokens_) { step_full = true; break; }
    seen.insert(r.ctx);
    tokens += r.k + 1;
    take.push_back(i);
  }
  std::vector<uint64_t> out;
  if (take.empty()) return out;
  // static batching waits for its fixed number of requests - unless the step cannot hold more anyway
  if (policy_ == kBatchStatic && !flush && !step_full && static_cast<int32_t>(take.size()) < batch_size_) return out;
  out.reserve(take.size());
  for (size_t i : take) out.push_back(q_[i].ticket);
  for (size_t j = take.size(); j-- > 0;) q_.erase(q_.begin() + static_cast<std::ptrdiff_t>(take[j]));
  return out;
}

// ---------------------------------------------------------------------------------------------
// Cut of a step's requests into attention work items (request, KV head, chunk of keys): the chunk length per
// request.  Every request is cut into equal parts.  Candidates are the one-wave plan (few requests: every item
// resident at once, parts in proportion to a request's cost - key tiles, weighted up when it has more than 16 or 32
// query rows, whose tiles take the tensor pipes longer - so that all blocks end together) and plans of several waves,
// which the hardware hands out as blocks retire; a small model of that picks among them.
void plan_attention_chunks(const int64_t* n_keys, const int32_t* q_tokens, int B, int Hkv, int group, int64_t slots,
                           bool uniform_tiles, int64_t part_rows_cap, int64_t* chunk_out, double* cost_out) {
  std::vector<int64_t> chunk_of(B, 256);
  std::vector<double> cost(B);
  // the warp-level kernel's tiles take the tensor pipes longer when a request has more than 32 query rows
  auto heavy = [&](int i) { return !uniform_tiles && q_tokens[i] * group > 32; };
  for (int i = 0; i < B; ++i) {
    const double passes = uniform_tiles ? 1.0 : (q_tokens[i] * group + 63) / 64;
    // time per key tile by query rows, from per-block timestamps inside a B=16 step: 1.0 us with up to 16 rows (memory
    // paces those blocks), 1.15 with up to 32, 1.93 with more (each warp then takes all 64 keys of a tile)
    const int rows = q_tokens[i] * group;
    const double per_tile = uniform_tiles ? 1.0 : rows > 32 ? 1.93 : rows > 16 ? 1.15 : 1.0;
    cost[i] = static_cast<double>((n_keys[i] + 63) / 64) * passes * per_tile;
  }
  auto part_rows_of = [&]() {
    int64_t rows = 0;
    for (int i = 0; i < B; ++i) {
      const int64_t nc = (n_keys[i] + chunk_of[i] - 1) / chunk_of[i];
      if (nc > 1) rows += nc * q_tokens[i];
    }
    return rows;
  };
  // How the items of a plan end on the resident blocks, by a small model: they are handed out longest first as blocks
  // retire; an item costs its key tiles (weighted as above) plus a fixed part worth about six tiles when its request
  // is cut (set-up, partial results, their merge) and three when it is not - the figures that make the model follow
  // the measured launch times at 64 and 128 requests (2048 against 4096 keys: 0.47 against 0.57 ms).
  {
    auto parts_for = [&](double per_item, std::vector<int64_t>& out) {   // parts of about per_item cost each
      int64_t items = 0;
      for (int i = 0; i < B; ++i) {
        const int64_t tiles = (n_keys[i] + 63) / 64;
        const int64_t nc = std::max<int64_t>(1, std::min<int64_t>(static_cast<int64_t>(std::ceil(cost[i] / per_item)),
                                                                  std::max<int64_t>(1, tiles / 2)));
        out[i] = (tiles + nc - 1) / nc * 64;
        items += (n_keys[i] + out[i] - 1) / out[i] * Hkv;
      }
      return items;
    };
    auto end_time = [&](const std::vector<int64_t>& chunks) {
      std::vector<std::pair<bool, double>> c;   // (heavy, cost)
      for (int i = 0; i < B; ++i) {
        const int64_t nc = (n_keys[i] + chunks[i] - 1) / chunks[i];
        for (int64_t j = 0; j < nc; ++j) {
          const int64_t cnt = std::min<int64_t>(chunks[i], n_keys[i] - j * chunks[i]);
          const double w = cost[i] * cnt / static_cast<double>(n_keys[i]) + (nc > 1 ? 6.0 : 3.0);
          c.emplace_back(heavy(i), w);   // stands for the Hkv equal items of this part: they start side by side
        }
      }
      std::sort(c.begin(), c.end(), [](const auto& x, const auto& y) { return x.first != y.first ? x.first : x.second > y.second; });
      std::priority_queue<double, std::vector<double>, std::greater<double>> free_at;
      for (int64_t k = 0; k < std::max<int64_t>(1, slots / Hkv); ++k) free_at.push(0.0);
      double end = 0.0;
      for (const auto& it : c) {
        const double t = free_at.top() + it.second;
        free_at.pop();
        free_at.push(t);
        end = std::max(end, t);
      }
      return end;
    };
    double best = -1.0;
    if (static_cast<int64_t>(B) * Hkv <= slots) {
      // one wave: the smallest cost per item for which the items still fit the slots (bisection on a monotone count)
      auto chunks_at = [&](int i, double per_item) {
        const int64_t tiles = (n_keys[i] + 63) / 64;
        const int64_t want = static_cast<int64_t>(std::ceil(cost[i] / per_item));
        return std::max<int64_t>(1, std::min(want, std::max<int64_t>(1, tiles / 2)));   // chunks of at least 2 tiles
      };
      auto items_at = [&](double per_item) {
        int64_t n = 0;
        for (int i = 0; i < B; ++i) n += chunks_at(i, per_item) * Hkv;
        return n;
      };
      double lo = 1.0, hi = 1.0;
      for (int i = 0; i < B; ++i) hi = std::max(hi, cost[i]);
      for (int it = 0; it < 30 && items_at(lo) > slots; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (items_at(mid) > slots) lo = mid; else hi = mid;
      }
      double per_item = items_at(lo) <= slots ? lo : hi;
      for (;;) {
        for (int i = 0; i < B; ++i) {
          const int64_t tiles = (n_keys[i] + 63) / 64;
          const int64_t nc = chunks_at(i, per_item);
          chunk_of[i] = (tiles + nc - 1) / nc * 64;
        }
        if (part_rows_of() <= part_rows_cap) break;
        per_item *= 1.5;   // fewer, longer chunks until the partial results fit
      }
      best = end_time(chunk_of);
    }
    // several waves: every request in equal parts of about one cost; the candidate that ends soonest wins (with few
    // requests that is the one-wave plan up to about 24 of them; at 32 - 36 the uncut requests of one wave differ too
    // much in length: 0.33 -> 0.29 and 0.47 -> 0.31 ms of attention in a 4-layer step)
    std::vector<int64_t> trial(B);
    double max_cost = 1.0;
    for (int i = 0; i < B; ++i) max_cost = std::max(max_cost, cost[i]);
    for (double per_item = 4.0;; per_item *= 2.0) {   // from 256 keys on (a finer grid measured no better)
      const bool whole = per_item >= max_cost;           // nobody is split any more: the last candidate
      const int64_t items = parts_for(whole ? max_cost : per_item, trial);
      std::swap(trial, chunk_of);
      const bool fits = part_rows_of() <= part_rows_cap;
      std::swap(trial, chunk_of);
      if (fits && (items <= 4 * slots || whole)) {
        const double end = end_time(trial);
        if (best < 0.0 || end < best) { best = end; chunk_of = trial; }
      }
      if (whole) break;
    }
  }
  for (int i = 0; i < B; ++i) {
    chunk_out[i] = chunk_of[i];
    if (cost_out) cost_out[i] = cost[i];
  }
}

}  // namespace sled

// ------------------------------------------------------------------ C face --
struct sled_planner {
  sled::Planner p;
  sled_planner(int policy, int32_t bs, int32_t mb, int32_t mt) : p(policy, bs, mb, mt) {}
};

extern "C" {

sled_planner* sled_planner_create(int32_t policy, int32_t batch_size, int32_t max_batch, int32_t max_step_tokens) {
  sled_planner* p = new sled_planner(policy, batch_size, max_batch, max_step_tokens);
  if (!p->p.valid()) {
    delete p;
    return nullptr;
  }
  return p;
}

void sled_planner_destroy(sled_planner* p) { delete p; }

int sled_planner_push(sled_planner* p, uint64_t ticket, uint64_t ctx_id, int32_t k) {
  return p ? p->p.push(ticket, ctx_id, k) : SLED_ERR_ARG;
}

int32_t sled_planner_next_batch(sled_planner* p, int32_t flush, uint64_t* tickets_out, int32_t cap) {
  if (!p || !tickets_out || cap <= 0) return SLED_ERR_ARG;
  // a batch is handed out whole or not at all
  sled::Planner probe = p->p;
  std::vector<uint64_t> b = probe.next_batch(flush != 0);
  if (static_cast<int32_t>(b.size()) > cap) return SLED_ERR_BATCH_TOO_LARGE;
  p->p = probe;
  std::copy(b.begin(), b.end(), tickets_out);
  return static_cast<int32_t>(b.size());
}

int32_t sled_planner_queued(sled_planner* p) { return p ? p->p.queued() : SLED_ERR_ARG; }

int sled_debug_plan_attention(const int64_t* n_keys, const int32_t* q_tokens, int32_t n_reqs, int32_t n_kv_heads,
                              int32_t group, int32_t resident_blocks, int64_t part_rows_cap, int64_t* chunk_keys_out) {
  if (!n_keys || !q_tokens || !chunk_keys_out || n_reqs <= 0 || n_kv_heads <= 0 || group <= 0 || resident_blocks <= 0 ||
      part_rows_cap < 0)
    return SLED_ERR_ARG;
  for (int i = 0; i < n_reqs; ++i)
    if (n_keys[i] <= 0 || q_tokens[i] <= 0) return SLED_ERR_ARG;
  sled::plan_attention_chunks(n_keys, q_tokens, n_reqs, n_kv_heads, group, resident_blocks, false, part_rows_cap,
                              chunk_keys_out, nullptr);
  return SLED_OK;
}

}  // extern "C"

#include "planner.h"

#include <algorithm>
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

}  // extern "C"

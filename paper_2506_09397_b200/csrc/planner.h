// Request queue and batch planner of the verification server (host only).
//
// Section 3.4 of the paper: verification requests of many devices wait in a queue; a batch planner takes
// requests out of it and hands one batch to the target model.  The paper's implementation is static batching
// (wait until a fixed number of requests is there); continuous batching (run whatever has arrived, up to the
// step's capacity) is the variant this library serves with by default.  The paper pads the requests of a batch
// to a common length; here a batch is ragged, so the capacity of a step is counted in tokens, sum (k_i + 1).
#pragma once
#include <cstdint>
#include <deque>
#include <vector>

namespace sled {

enum BatchPolicy { kBatchStatic = 0, kBatchContinuous = 1 };

struct QueuedRequest {
  uint64_t ticket;
  uint64_t ctx;
  int32_t k;
};

class Planner {
 public:
  // batch_size: requests a static batch waits for (ignored by the continuous policy);
  // max_batch / max_step_tokens: the most requests / tokens one step can take
  Planner(int policy, int32_t batch_size, int32_t max_batch, int32_t max_step_tokens);
  bool valid() const { return valid_; }
  int push(uint64_t ticket, uint64_t ctx, int32_t k);
  // Takes the next batch out of the queue, in arrival order; returns its tickets.  A request whose context is
  // already in the batch stays queued, in place (one context is verified at most once per step).  A request that
  // does not fit the step's remaining tokens ends the batch (later requests do not overtake it).
  //   static:      nothing while fewer than batch_size requests of distinct contexts wait, unless flush;
  //                never more than batch_size
  //   continuous:  whatever is there, up to max_batch
  std::vector<uint64_t> next_batch(bool flush);
  int32_t queued() const { return static_cast<int32_t>(q_.size()); }
  int policy() const { return policy_; }

 private:
  int policy_;
  int32_t batch_size_, max_batch_, max_step_tokens_;
  bool valid_;
  std::deque<QueuedRequest> q_;
};

// The cut of a step's requests into attention work items: chunk_out[i] = keys per item of request i (a multiple of
// 64; the request has ceil(n_keys[i] / chunk_out[i]) items per KV head).  n_keys[i]: keys request i attends to,
// q_tokens[i]: its query tokens (k + 1), group: query heads per KV head, slots: blocks resident at once,
// uniform_tiles: every key tile costs the same whatever the number of query rows (the tcgen05 kernel),
// part_rows_cap: most rows of partial results (one per chunk and query token of every request that is cut).
// cost_out (may be null): the cost the plan assigns to each whole request, in key tiles.
void plan_attention_chunks(const int64_t* n_keys, const int32_t* q_tokens, int B, int Hkv, int group, int64_t slots,
                           bool uniform_tiles, int64_t part_rows_cap, int64_t* chunk_out, double* cost_out);

}  // namespace sled

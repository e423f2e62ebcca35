// Host-side bookkeeping of the paged KV cache: which context owns which pages, how
// many tokens are cached, which token is pending.  No device code: verification
// reserves slots for k+1 new tokens before the forward pass, then keeps the accepted
// prefix and gives back pages that ended up empty (commit / rollback by truncation).
#pragma once
#include <cstdint>
#include <unordered_map>
#include <vector>

namespace sled {

struct CtxState {
  int64_t n_kv = 0;        // tokens whose keys/values are kept
  int64_t n_reserved = 0;  // slots reserved behind them for the step in flight
  int32_t pending = 0;     // last committed token; its KV is written by the next step
  std::vector<int32_t> pages;
  // committed tokens from sequence index hist_start on (the last one is `pending`): what a request's base_len can go
  // back to.  A context opened from cache content alone knows its history from the pending token on.
  std::vector<int32_t> hist;
  int64_t hist_start = 0;
};

class KvManager {
 public:
  KvManager(int32_t n_pages, int32_t page_size);
  int open(uint64_t ctx, int64_t n_kv, int32_t pending);
  // base_len (may be null; entries of 0 mean "continue at the end"): request i continues the first base_len[i]
  // committed tokens of its context, which is cut back to that length before slots are reserved
  int reserve_batch(const uint64_t* ctxs, const int32_t* extra, int32_t n, const int64_t* base_len = nullptr);
  // kept: the n_keep - 1 tokens behind the old pending one whose cache entries stay (null: unknown, the history
  // restarts at the new pending token)
  int commit(uint64_t ctx, int32_t n_keep, int32_t pending, const int32_t* kept = nullptr);
  int truncate(uint64_t ctx, int64_t n_kv, int32_t pending);
  int release(uint64_t ctx);
  void shuffle_free(uint64_t seed);  // seeded permutation of the free list
  const CtxState* find(uint64_t ctx) const;
  int32_t free_pages() const { return static_cast<int32_t>(free_.size()); }
  int32_t total_pages() const { return n_pages_; }
  int32_t page_size() const { return page_size_; }
  int32_t open_contexts() const { return static_cast<int32_t>(ctx_.size()); }
  // physical slot (page * page_size + offset) of a context's token index
  int64_t slot_of(const CtxState& c, int64_t token_index) const {
    return static_cast<int64_t>(c.pages[token_index / page_size_]) * page_size_ + token_index % page_size_;
  }

 private:
  int64_t pages_for(int64_t tokens) const { return (tokens + page_size_ - 1) / page_size_; }
  void shrink_to(CtxState& c, int64_t tokens);
  int32_t n_pages_, page_size_;
  std::vector<int32_t> free_;  // stack of free page ids
  std::unordered_map<uint64_t, CtxState> ctx_;
};

}  // namespace sled

#include "kv_manager.h"

#include <unordered_set>
#include <utility>

#include "../../include/sled.h"

namespace sled {

KvManager::KvManager(int32_t n_pages, int32_t page_size) : n_pages_(n_pages), page_size_(page_size) {
  free_.reserve(n_pages);
  for (int32_t p = n_pages - 1; p >= 0; --p) free_.push_back(p);  // page 0 is handed out first
}

const CtxState* KvManager::find(uint64_t ctx) const {
  auto it = ctx_.find(ctx);
  return it == ctx_.end() ? nullptr : &it->second;
}

void KvManager::shrink_to(CtxState& c, int64_t tokens) {
  const int64_t keep = pages_for(tokens);
  while (static_cast<int64_t>(c.pages.size()) > keep) {
    free_.push_back(c.pages.back());
    c.pages.pop_back();
  }
}

int KvManager::open(uint64_t ctx, int64_t n_kv, int32_t pending) {
  if (n_kv < 0) return SLED_ERR_ARG;
  if (ctx_.count(ctx)) return SLED_ERR_DUP_CTX;
  const int64_t need = pages_for(n_kv);
  if (need > static_cast<int64_t>(free_.size())) return SLED_ERR_NO_PAGES;
  CtxState c;
  c.n_kv = n_kv;
  c.pending = pending;
  c.hist_start = n_kv;
  c.hist.assign(1, pending);
  for (int64_t i = 0; i < need; ++i) {
    c.pages.push_back(free_.back());
    free_.pop_back();
  }
  ctx_.emplace(ctx, std::move(c));
  return SLED_OK;
}

int KvManager::reserve_batch(const uint64_t* ctxs, const int32_t* extra, int32_t n, const int64_t* base_len) {
  // first pass: everything that can fail, without touching any state
  std::unordered_set<uint64_t> seen;
  int64_t need = 0;
  for (int32_t i = 0; i < n; ++i) {
    if (extra[i] < 0) return SLED_ERR_ARG;
    if (!seen.insert(ctxs[i]).second) return SLED_ERR_DUP_CTX;
    auto it = ctx_.find(ctxs[i]);
    if (it == ctx_.end()) return SLED_ERR_UNKNOWN_CTX;
    const CtxState& c = it->second;
    int64_t n_kv = c.n_kv;
    if (base_len && base_len[i] != 0) {
      // only as far back as the tokens are known, and never beyond the current end
      if (base_len[i] < c.hist_start + 1 || base_len[i] > c.n_kv + 1) return SLED_ERR_BASE_LEN;
      n_kv = base_len[i] - 1;
    }
    need += pages_for(n_kv + extra[i]) - static_cast<int64_t>(c.pages.size());   // negative: pages come back
  }
  if (need > static_cast<int64_t>(free_.size())) return SLED_ERR_NO_PAGES;
  if (base_len)   // contexts that shrink first, so that their pages are there for the ones that grow
    for (int32_t i = 0; i < n; ++i) {
      if (base_len[i] == 0) continue;
      CtxState& c = ctx_.find(ctxs[i])->second;
      c.n_kv = base_len[i] - 1;
      c.hist.resize(static_cast<size_t>(base_len[i] - c.hist_start));
      c.pending = c.hist.back();
      shrink_to(c, c.n_kv + extra[i]);
    }
  for (int32_t i = 0; i < n; ++i) {
    CtxState& c = ctx_.find(ctxs[i])->second;
    const int64_t want = pages_for(c.n_kv + extra[i]);
    while (static_cast<int64_t>(c.pages.size()) < want) {
      c.pages.push_back(free_.back());
      free_.pop_back();
    }
    c.n_reserved = extra[i];
  }
  return SLED_OK;
}

int KvManager::commit(uint64_t ctx, int32_t n_keep, int32_t pending, const int32_t* kept) {
  auto it = ctx_.find(ctx);
  if (it == ctx_.end()) return SLED_ERR_UNKNOWN_CTX;
  CtxState& c = it->second;
  if (n_keep < 0 || n_keep > c.n_reserved) return SLED_ERR_ARG;
  c.n_kv += n_keep;
  c.n_reserved = 0;
  c.pending = pending;
  if (n_keep == 0) {
    c.hist.back() = pending;   // nothing kept: the pending token stays (callers pass the old one back)
  } else if (kept || n_keep == 1) {
    for (int32_t j = 0; j + 1 < n_keep; ++j) c.hist.push_back(kept[j]);
    c.hist.push_back(pending);
  } else {                     // tokens not given: what is known restarts at the new pending token
    c.hist_start = c.n_kv;
    c.hist.assign(1, pending);
  }
  shrink_to(c, c.n_kv);
  return SLED_OK;
}

int KvManager::truncate(uint64_t ctx, int64_t n_kv, int32_t pending) {
  auto it = ctx_.find(ctx);
  if (it == ctx_.end()) return SLED_ERR_UNKNOWN_CTX;
  CtxState& c = it->second;
  if (n_kv < 0 || n_kv > c.n_kv) return SLED_ERR_ARG;
  c.n_kv = n_kv;
  c.n_reserved = 0;
  c.pending = pending;
  if (n_kv >= c.hist_start && c.hist[static_cast<size_t>(n_kv - c.hist_start)] == pending) {
    c.hist.resize(static_cast<size_t>(n_kv - c.hist_start) + 1);   // a cut inside the known history
  } else {
    c.hist_start = n_kv;
    c.hist.assign(1, pending);
  }
  shrink_to(c, c.n_kv);
  return SLED_OK;
}

int KvManager::release(uint64_t ctx) {
  auto it = ctx_.find(ctx);
  if (it == ctx_.end()) return SLED_ERR_UNKNOWN_CTX;
  shrink_to(it->second, 0);
  ctx_.erase(it);
  return SLED_OK;
}

void KvManager::shuffle_free(uint64_t seed) {
  uint64_t state = seed * 0x9E3779B97F4A7C15ull + 0xD1B54A32D192ED03ull;
  auto next = [&state]() {  // splitmix64
    uint64_t z = (state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  };
  for (size_t i = free_.size(); i > 1; --i) std::swap(free_[i - 1], free_[next() % i]);
}

}  // namespace sled

// ------------------------------------------------------------------ C face --
struct sled_kvm {
  sled::KvManager m;
  sled_kvm(int32_t n, int32_t p) : m(n, p) {}
};

extern "C" {

sled_kvm* sled_kvm_create(int32_t n_pages, int32_t page_size) {
  if (n_pages <= 0 || page_size <= 0) return nullptr;
  return new sled_kvm(n_pages, page_size);
}

void sled_kvm_destroy(sled_kvm* m) { delete m; }

int sled_kvm_open(sled_kvm* m, uint64_t ctx_id, int64_t n_kv, int32_t pending) {
  return m ? m->m.open(ctx_id, n_kv, pending) : SLED_ERR_ARG;
}

int sled_kvm_reserve_batch(sled_kvm* m, const uint64_t* ctx_ids, const int32_t* extra, int32_t n) {
  if (!m || n < 0 || (n > 0 && (!ctx_ids || !extra))) return SLED_ERR_ARG;
  return m->m.reserve_batch(ctx_ids, extra, n);
}

int sled_kvm_commit(sled_kvm* m, uint64_t ctx_id, int32_t n_keep, int32_t pending) {
  return m ? m->m.commit(ctx_id, n_keep, pending) : SLED_ERR_ARG;
}

int sled_kvm_reserve_batch_at(sled_kvm* m, const uint64_t* ctx_ids, const int32_t* extra, const int64_t* base_len,
                              int32_t n) {
  if (!m || n < 0 || (n > 0 && (!ctx_ids || !extra))) return SLED_ERR_ARG;
  if (base_len)
    for (int32_t i = 0; i < n; ++i)
      if (base_len[i] < 0) return SLED_ERR_ARG;
  return m->m.reserve_batch(ctx_ids, extra, n, base_len);
}

int sled_kvm_commit_tokens(sled_kvm* m, uint64_t ctx_id, int32_t n_keep, int32_t pending, const int32_t* kept) {
  if (!m || (n_keep > 1 && !kept)) return SLED_ERR_ARG;
  return m->m.commit(ctx_id, n_keep, pending, kept);
}

int sled_kvm_history(sled_kvm* m, uint64_t ctx_id, int64_t* hist_start, int32_t* n_tokens, int32_t* tokens_out,
                     int32_t cap) {
  if (!m) return SLED_ERR_ARG;
  const sled::CtxState* c = m->m.find(ctx_id);
  if (!c) return SLED_ERR_UNKNOWN_CTX;
  if (hist_start) *hist_start = c->hist_start;
  if (n_tokens) *n_tokens = static_cast<int32_t>(c->hist.size());
  if (tokens_out)
    for (int32_t i = 0; i < cap && i < static_cast<int32_t>(c->hist.size()); ++i) tokens_out[i] = c->hist[i];
  return SLED_OK;
}

int sled_kvm_release(sled_kvm* m, uint64_t ctx_id) { return m ? m->m.release(ctx_id) : SLED_ERR_ARG; }

int sled_kvm_query(sled_kvm* m, uint64_t ctx_id, int64_t* n_kv, int32_t* pending, int32_t* n_pages,
                   int32_t* pages_out, int32_t cap) {
  if (!m) return SLED_ERR_ARG;
  const sled::CtxState* c = m->m.find(ctx_id);
  if (!c) return SLED_ERR_UNKNOWN_CTX;
  if (n_kv) *n_kv = c->n_kv;
  if (pending) *pending = c->pending;
  if (n_pages) *n_pages = static_cast<int32_t>(c->pages.size());
  if (pages_out)
    for (int32_t i = 0; i < cap && i < static_cast<int32_t>(c->pages.size()); ++i) pages_out[i] = c->pages[i];
  return SLED_OK;
}

int32_t sled_kvm_free_pages(sled_kvm* m) { return m ? m->m.free_pages() : -1; }

int sled_kvm_pack(sled_kvm* m, const uint64_t* ctx_ids, const int32_t* k, const int32_t* const* drafts, int32_t n,
                  int32_t* cu_q, int32_t* ids, int32_t* tok_req, int32_t* tok_pos, int32_t* tok_slot) {
  if (!m || n < 0 || !cu_q) return SLED_ERR_ARG;
  int32_t t = 0;
  cu_q[0] = 0;
  for (int32_t i = 0; i < n; ++i) {
    const sled::CtxState* c = m->m.find(ctx_ids[i]);
    if (!c) return SLED_ERR_UNKNOWN_CTX;
    if (k[i] < 0 || k[i] + 1 > c->n_reserved) return SLED_ERR_K_RANGE;
    for (int32_t j = 0; j <= k[i]; ++j, ++t) {
      ids[t] = j == 0 ? c->pending : drafts[i][j - 1];
      tok_req[t] = i;
      tok_pos[t] = static_cast<int32_t>(c->n_kv + j);
      tok_slot[t] = static_cast<int32_t>(m->m.slot_of(*c, c->n_kv + j));
    }
    cu_q[i + 1] = t;
  }
  return SLED_OK;
}

}  // extern "C"

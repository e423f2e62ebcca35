// Engine behind the C boundary: owns weights, the paged KV pool and the step workspaces,
// packs a ragged batch, issues the kernel sequence of one verification step and commits
// or rolls back the cache afterwards.  Host logic only; kernels live in the other files.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <queue>
#include <vector>

#include "../../include/sled.h"
#include "gemm_tc.h"
#include "kernels.h"
#include "kv_manager.h"
#include "planner.h"

#include <unordered_map>

using namespace sled;

namespace {

#define CU_TRY(expr)                                                            \
  do {                                                                          \
    cudaError_t err__ = (expr);                                                 \
    if (err__ != cudaSuccess) {                                                 \
      std::fprintf(stderr, "sled: %s failed: %s (%s:%d)\n", #expr, cudaGetErrorString(err__), __FILE__, __LINE__); \
      return SLED_ERR_DEVICE;                                                   \
    }                                                                           \
  } while (0)

size_t dtype_size(int dt) { return dt == SLED_BF16 ? 2 : 4; }
size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Linear {      // one weight matrix [N][K] in device memory
  void* w = nullptr;
  float* scale = nullptr;   // 8-bit weights: one scale per output row
  int N = 0, K = 0;
  TcWeight tc;       // tensor-core operand description (bf16 and 8-bit weights)
};

struct Layer {
  void* attn_norm;
  void* ffn_norm;
  Linear qkv, o, gate_up, down;
};

struct PlanReq {     // tokens fed for one context in one forward pass
  uint64_t ctx;
  const int32_t* toks;
  int n;
};

enum Kind { K_LINEAR = 0, K_ATTN = 1, K_ACCEPT = 2, K_OTHER = 3, K_KINDS = 4 };

constexpr int kResultsHead = 4;   // words in front of the per-request results: [0] = device error word

}  // namespace

struct sled_engine {
  sled_config cfg;
  int n_sm = 0;
  cudaStream_t stream = nullptr, copy_stream = nullptr;
  bool own_stream = false;
  cudaEvent_t ev_copy = nullptr, ev_a = nullptr, ev_b = nullptr;
  KvManager* kvm = nullptr;
  bool commit = true;
  long long probe_wait_cycles = 0;   // > 0: the next verification step starts with the give-up self-test kernel
  int timing = 0;   // 0 off, 1 device timestamps per launch (overlap untouched), 2 events between kernel groups (serialises)

  // device memory
  std::vector<void*> allocs;
  void* tok_emb = nullptr;
  void* final_norm = nullptr;
  Linear lm_head;
  std::vector<Layer> layers;
  char* kpool = nullptr;
  char* vpool = nullptr;
  size_t kv_layer_bytes = 0;
  std::vector<CUtensorMap> kv_maps;  // [2 * layer + {0: K, 1: V}] for the tensor-core attention kernel
  float* x = nullptr;
  void* act_norm = nullptr;
  void* q_buf = nullptr;
  void* attn_out = nullptr;
  void* act_ffn = nullptr;
  float* partial = nullptr;
  size_t partial_elems = 0;
  float* logits = nullptr;
  float2* rope_cs = nullptr;
  float* part_acc = nullptr;
  float* part_ml = nullptr;
  int part_rows_cap = 0;
  float* q_stage = nullptr;
  bool attn_tc = false;          // head_dim 128, bf16 cache, 16-token pages: attention may run on tcgen05
  TcActivation tc_norm, tc_attn, tc_ffn;
  TcActivation8 a8_norm, a8_attn, a8_ffn;   // 8-bit weights: the same activations as two e4m3 parts + token scales
  bool norm_split = false;                  // the normalisation kernel has filled a8_norm for the act_norm now in place
  bool attn_split = false;                  // the same for a8_attn and the attention output
  int32_t* tc_error = nullptr;  // device word set by a kernel whose bounded wait ran out: the first word of the
                                // results block (d_results), so the step's one result copy brings it along

  // step metadata: pinned staging + device mirror
  char* h_meta = nullptr;
  char* d_meta = nullptr;
  size_t meta_cap = 0, meta_used = 0;
  int32_t* h_results = nullptr;
  int32_t* d_results = nullptr;
  int last_T = 0;

  // timing
  std::vector<cudaEvent_t> ev_pool;
  std::vector<int> ev_kind;
  size_t ev_used = 0;
  unsigned long long* d_stamps = nullptr;   // [2][stamp_cap]: begin times, then end times
  unsigned long long* h_stamps = nullptr;   // pinned mirror
  std::vector<int> stamp_kind;
  size_t stamp_cap = 0, stamp_used = 0;

  // server loop (sled_submit / sled_step / sled_poll): queued requests with their own copy of the draft tokens,
  // finished results by ticket
  struct Waiting {
    sled_request req;
    std::vector<int32_t> drafts;
  };
  Planner* planner = nullptr;
  std::unordered_map<uint64_t, Waiting> waiting;
  std::unordered_map<uint64_t, sled_result> finished;
  uint64_t next_ticket = 1;

  sled_stats st{};
  int64_t launches_step = 0;
  int lin_launches = 0, attn_launches = 0;

  int adtype() const { return cfg.weight_dtype; }  // activations fed to linear layers follow the weights

  template <typename T> T* meta_alloc(size_t count, T** dev) {
    size_t off = align_up(meta_used, 16);
    size_t bytes = count * sizeof(T);
    if (off + bytes > meta_cap) return nullptr;
    meta_used = off + bytes;
    *dev = reinterpret_cast<T*>(d_meta + off);
    return reinterpret_cast<T*>(h_meta + off);
  }

  Stamp stamp(int kind) {  // timing mode 1: the next launch's pair of timestamp words
    Stamp st;
    if (timing != 1 || stamp_used >= stamp_cap) return st;
    st.begin = d_stamps + stamp_used;
    st.end = d_stamps + stamp_cap + stamp_used;
    stamp_kind[stamp_used++] = kind;
    return st;
  }
  void mark(int kind) {  // timing mode 2: an event before every kernel group, tagged with what follows
    if (timing != 2 || ev_used >= ev_pool.size()) return;
    cudaEventRecord(ev_pool[ev_used], stream);
    ev_kind[ev_used] = kind;
    ++ev_used;
  }
  void count(int n, int kind) {
    if (n > 0) {
      launches_step += n;
      if (kind == K_LINEAR) lin_launches += n;
      if (kind == K_ATTN) attn_launches += n;
    }
  }
};

namespace {

int dmalloc(sled_engine* e, void** p, size_t bytes) {
  if (bytes == 0) bytes = 16;
  cudaError_t err = cudaMalloc(p, bytes);
  if (err != cudaSuccess) {
    std::fprintf(stderr, "sled: cudaMalloc(%zu) failed: %s\n", bytes, cudaGetErrorString(err));
    *p = nullptr;
    return SLED_ERR_DEVICE;
  }
  e->allocs.push_back(*p);
  return SLED_OK;
}

// split-K factor of a linear layer on the CUDA-core path: fill the machine when there are few output tiles
int simt_split(int T, int N, int K, int n_sm) {
  const int blocks = ((N + 63) / 64) * ((T + 31) / 32);
  int s = 1;
  if (blocks < 2 * n_sm) s = (2 * n_sm + blocks - 1) / blocks;
  s = std::min(s, std::max(1, K / 256));
  return std::max(1, std::min(s, 8));
}

int linear_split(const sled_engine* e, int T, const Linear& L) {
  if (L.tc.f8) return tc_gemm_split_f8(T, L.N, L.K, e->n_sm);
  if (e->cfg.weight_dtype == SLED_BF16) return tc_gemm_split(T, L.N, L.K, e->n_sm);
  return simt_split(T, L.N, L.K, e->n_sm);
}

// out partial sums [split][T][N] into e->partial (or into `dst` when given, then split must be 1)
int run_linear(sled_engine* e, const void* A, const TcActivation* tcA, const Linear& L, int T, float* dst, int* split_out,
               const TcEpilogue& epi = TcEpilogue()) {
  int split = dst ? 1 : linear_split(e, T, L);
  float* out = dst ? dst : e->partial;
  const int64_t stride = static_cast<int64_t>(T) * L.N;
  if (!dst && static_cast<size_t>(split) * stride > e->partial_elems) return SLED_ERR_DEVICE;
  const TcActivation8* a8 = nullptr;
  if (L.tc.f8) {   // fp8 MMAs: the input goes in as two e4m3 parts per element and a scale per token
    a8 = tcA == &e->tc_norm ? &e->a8_norm : tcA == &e->tc_attn ? &e->a8_attn : &e->a8_ffn;
    if (!(a8 == &e->a8_norm && e->norm_split) && !(a8 == &e->a8_attn && e->attn_split)) {
      e->mark(K_OTHER);
      const Stamp ss = e->stamp(K_OTHER);
      const int ns = tc_split_rows_launch(A, T, *a8, e->stream, ss.begin, ss.end);
      if (ns < 0) return SLED_ERR_DEVICE;
      e->count(ns, K_OTHER);
    }
  }
  e->mark(K_LINEAR);
  const Stamp st = e->stamp(K_LINEAR);
  int n;
  if (e->cfg.weight_dtype == SLED_BF16) {
    TcEpilogue ep = epi;
    ep.stamp_begin = st.begin;
    ep.stamp_end = st.end;
    n = a8 ? tc_gemm_f8_launch(*a8, L.tc, T, split, out, stride, e->tc_error, ep, e->stream)
           : tc_gemm_launch(*tcA, L.tc, T, split, out, stride, e->tc_error, ep, e->stream);
  } else {
    n = launch_gemm_simt(A, e->adtype(), L.w, e->cfg.weight_dtype, T, L.N, L.K, split, out, stride, e->stream, st);
  }
  if (n < 0) return SLED_ERR_DEVICE;
  e->count(n, K_LINEAR);
  *split_out = split;
  return SLED_OK;
}

struct Packed {
  int T = 0, B = 0;
  int32_t *ids, *tok_req, *tok_pos, *tok_slot, *tok_part, *cu_q, *kv_base, *pt_off, *req_chunks, *req_chunk_keys, *page_table;
  int4* items;
  int n_items = 0;
  bool any_split = false;
  bool use_tc = false;   // the tcgen05 attention kernel serves this step (every request has at most 48 query rows)
  // host views
  int32_t *h_cu_q, *h_kv_base;
};

// Builds the ragged description of a step in the pinned staging area.  `base_shift`: tokens of the
// request that are already cached (attention-only entry: the last q_len cached tokens act as new ones).
int pack_step(sled_engine* e, const std::vector<PlanReq>& plan, bool already_cached, Packed* pk) {
  const int B = static_cast<int>(plan.size());
  int T = 0;
  for (auto& r : plan) T += r.n;
  pk->T = T;
  pk->B = B;
  const int ps = e->cfg.page_size, Hkv = e->cfg.n_kv_heads;
  int32_t* h_ids = e->meta_alloc<int32_t>(T, &pk->ids);
  int32_t* h_req = e->meta_alloc<int32_t>(T, &pk->tok_req);
  int32_t* h_pos = e->meta_alloc<int32_t>(T, &pk->tok_pos);
  int32_t* h_slot = e->meta_alloc<int32_t>(T, &pk->tok_slot);
  int32_t* h_part = e->meta_alloc<int32_t>(T, &pk->tok_part);
  int32_t* h_cu = e->meta_alloc<int32_t>(B + 1, &pk->cu_q);
  int32_t* h_base = e->meta_alloc<int32_t>(B, &pk->kv_base);
  int32_t* h_ptoff = e->meta_alloc<int32_t>(B + 1, &pk->pt_off);
  int32_t* h_chunks = e->meta_alloc<int32_t>(B, &pk->req_chunks);
  int32_t* h_chunk_keys = e->meta_alloc<int32_t>(B, &pk->req_chunk_keys);
  if (!h_chunk_keys) return SLED_ERR_BATCH_TOO_LARGE;
  if (!h_ids || !h_req || !h_pos || !h_slot || !h_part || !h_cu || !h_base || !h_ptoff || !h_chunks)
    return SLED_ERR_BATCH_TOO_LARGE;
  pk->h_cu_q = h_cu;
  pk->h_kv_base = h_base;

  int64_t total_pages = 0;
  std::vector<int64_t> n_keys(B);
  int t = 0;
  h_cu[0] = 0;
  h_ptoff[0] = 0;
  for (int i = 0; i < B; ++i) {
    const CtxState* c = e->kvm->find(plan[i].ctx);
    if (!c) return SLED_ERR_UNKNOWN_CTX;
    const int64_t base = already_cached ? c->n_kv - plan[i].n : c->n_kv;
    if (base < 0) return SLED_ERR_ARG;
    h_base[i] = static_cast<int32_t>(base);
    n_keys[i] = base + plan[i].n;
    for (int j = 0; j < plan[i].n; ++j, ++t) {
      h_ids[t] = plan[i].toks ? plan[i].toks[j] : 0;
      h_req[t] = i;
      h_pos[t] = static_cast<int32_t>(base + j);
      h_slot[t] = static_cast<int32_t>(e->kvm->slot_of(*c, base + j));
      h_part[t] = 0;
    }
    h_cu[i + 1] = t;
    const int64_t np = (n_keys[i] + ps - 1) / ps;
    total_pages += np;
    h_ptoff[i + 1] = static_cast<int32_t>(total_pages);
  }
  int32_t* h_pt = e->meta_alloc<int32_t>(static_cast<size_t>(total_pages), &pk->page_table);
  if (!h_pt) return SLED_ERR_BATCH_TOO_LARGE;
  for (int i = 0; i < B; ++i) {
    const CtxState* c = e->kvm->find(plan[i].ctx);
    const int np = h_ptoff[i + 1] - h_ptoff[i];
    std::memcpy(h_pt + h_ptoff[i], c->pages.data(), sizeof(int32_t) * np);
  }

  // Attention work items: (request, KV head, chunk of keys).  The chunk length is chosen per request: every request
  // is cut into equal parts.  Candidates are the one-wave plan (few requests: every item resident at once, two blocks
  // per SM, parts in proportion to a request's cost - key tiles, weighted up when it has more than 32 query rows,
  // whose tiles take the tensor pipes longer - so that all blocks end together) and plans of several waves, which
  // the hardware hands out as blocks retire; a small model of that picks among them (below).
  const int group = e->cfg.n_q_heads / Hkv;
  int max_rows = 0;
  for (int i = 0; i < B; ++i) max_rows = std::max(max_rows, plan[i].n * group);
  pk->use_tc = e->attn_tc && max_rows <= 48;
  // blocks resident at once: the tcgen05 kernel runs one block per SM, the warp-level kernel two
  const int64_t slots = (pk->use_tc ? 1LL : 2LL) * e->n_sm;
  std::vector<int64_t> chunk_of(B, 256);
  std::vector<double> cost(B);
  std::vector<int32_t> q_tokens(B);
  for (int i = 0; i < B; ++i) q_tokens[i] = plan[i].n;
  plan_attention_chunks(n_keys.data(), q_tokens.data(), B, Hkv, group, slots, pk->use_tc, e->part_rows_cap, chunk_of.data(),
                        cost.data());
  auto heavy = [&](int i) { return !pk->use_tc && plan[i].n * group > 32; };
  struct It { int req, kvh, start, count; double cost; bool heavy; };
  std::vector<It> its;
  int part_rows = 0;
  for (int i = 0; i < B; ++i) {
    const int64_t chunk = chunk_of[i];
    const int nc = static_cast<int>((n_keys[i] + chunk - 1) / chunk);
    h_chunks[i] = nc;
    h_chunk_keys[i] = static_cast<int32_t>(std::min<int64_t>(chunk, 1 << 30));
    if (nc > 1) {
      pk->any_split = true;
      for (int tt = h_cu[i]; tt < h_cu[i + 1]; ++tt) {
        h_part[tt] = part_rows;
        part_rows += nc;
      }
    }
    for (int c = 0; c < nc; ++c) {
      const int start = static_cast<int>(c * chunk);
      const int cnt = static_cast<int>(std::min<int64_t>(chunk, n_keys[i] - start));
      for (int kvh = 0; kvh < Hkv; ++kvh) its.push_back({i, kvh, start, cnt, cost[i] * cnt / static_cast<double>(n_keys[i]), heavy(i)});
    }
  }
  // heavy items first, then by cost: blocks are handed to the SMs in turn, so an SM's second block is a light one
  std::stable_sort(its.begin(), its.end(), [](const It& a, const It& b) {
    if (a.heavy != b.heavy) return a.heavy;
    return a.cost > b.cost;
  });
  int4* h_items = e->meta_alloc<int4>(its.size(), &pk->items);
  if (!h_items) return SLED_ERR_BATCH_TOO_LARGE;
  for (size_t i = 0; i < its.size(); ++i) h_items[i] = make_int4(its[i].req, its[i].kvh, its[i].start, its[i].count);
  pk->n_items = static_cast<int>(its.size());
  return SLED_OK;
}

AttnArgs attn_args(sled_engine* e, const Packed& pk, int layer, const void* q, void* out) {
  AttnArgs a{};
  a.items = pk.items;
  a.n_items = pk.n_items;
  a.q = q;
  a.out = out;
  a.kpool = e->kpool + e->kv_layer_bytes * layer;
  a.vpool = e->vpool + e->kv_layer_bytes * layer;
  a.cu_q = pk.cu_q;
  a.kv_base = pk.kv_base;
  a.page_table = pk.page_table;
  a.pt_off = pk.pt_off;
  a.tok_req = pk.tok_req;
  a.tok_part = pk.tok_part;
  a.req_chunks = pk.req_chunks;
  a.part_acc = pk.any_split ? e->part_acc : nullptr;
  a.part_ml = pk.any_split ? e->part_ml : nullptr;
  a.T = pk.T;
  a.Hq = e->cfg.n_q_heads;
  a.Hkv = e->cfg.n_kv_heads;
  a.h = e->cfg.head_dim;
  a.page_size = e->cfg.page_size;
  a.req_chunk_keys = pk.req_chunk_keys;
  a.adtype = e->adtype();
  a.kvdtype = e->cfg.kv_dtype;
  if (!e->kv_maps.empty()) {
    a.map_k = &e->kv_maps[2 * layer];
    a.map_v = &e->kv_maps[2 * layer + 1];
    a.error = e->tc_error;
  }
  a.use_tc = pk.use_tc ? 1 : 0;
  a.stamp = e->stamp(K_ATTN);
  if (pk.any_split) a.stamp_merge = e->stamp(K_ATTN);
  return a;
}

// The transformer forward over a packed step: embedding .. final norm (.. LM head).  Enqueue only.
int run_forward(sled_engine* e, const Packed& pk, bool need_logits) {
  const sled_config& c = e->cfg;
  const int T = pk.T, d = c.d_model, ad = e->adtype();
  const bool f8 = !e->layers.empty() && e->layers[0].qkv.tc.f8;   // fp8 linear layers: the normalisation also splits its output
  int n;
  e->mark(K_OTHER);
  n = launch_embed(e->tok_emb, c.weight_dtype, pk.ids, T, d, e->x, e->stream, e->stamp(K_OTHER));
  e->count(n, K_OTHER);
  n = launch_rope_table(pk.tok_pos, T, c.head_dim, c.rope_theta, e->rope_cs, e->stream, e->stamp(K_OTHER));
  e->count(n, K_OTHER);
  int split = 0;           // split count of the partial sums waiting to be added to x
  int64_t stride = 0;
  for (int l = 0; l < c.n_layers; ++l) {
    Layer& L = e->layers[l];
    e->mark(K_OTHER);
    n = launch_add_rmsnorm(e->x, e->partial, split, stride, L.attn_norm, c.weight_dtype, c.rms_eps, T, d, e->act_norm,
                           ad, e->stream, e->stamp(K_OTHER), f8 ? e->a8_norm.data : nullptr, e->a8_norm.rows,
                           f8 ? e->a8_norm.scale : nullptr, &e->norm_split);
    if (n < 0) return SLED_ERR_DEVICE;
    e->count(n, K_OTHER);
    int s_qkv;
    int rc = run_linear(e, e->act_norm, &e->tc_norm, L.qkv, T, nullptr, &s_qkv);
    if (rc) return rc;
    e->mark(K_OTHER);
    n = launch_rope_kv(e->partial, s_qkv, static_cast<int64_t>(T) * L.qkv.N, e->rope_cs, pk.tok_slot, T, c.n_q_heads,
                       c.n_kv_heads, c.head_dim, c.page_size, e->q_buf, ad, e->kpool + e->kv_layer_bytes * l,
                       e->vpool + e->kv_layer_bytes * l, c.kv_dtype, e->stream, e->stamp(K_OTHER));
    if (n < 0) return SLED_ERR_DEVICE;
    e->count(n, K_OTHER);
    e->mark(K_ATTN);
    AttnArgs aa = attn_args(e, pk, l, e->q_buf, e->attn_out);
    if (f8) {   // fp8 linear layers: the merge kernel also writes the attention output as two e4m3 parts per element
      aa.out8 = e->a8_attn.data;
      aa.out8_lo_row0 = e->a8_attn.rows;
      aa.out8_scale = e->a8_attn.scale;
    }
    n = launch_attention(aa, e->stream, &e->attn_split);
    if (n < 0) return SLED_ERR_DEVICE;
    e->count(n, K_ATTN);
    rc = run_linear(e, e->attn_out, &e->tc_attn, L.o, T, nullptr, &split);
    if (rc) return rc;
    stride = static_cast<int64_t>(T) * L.o.N;
    e->mark(K_OTHER);
    n = launch_add_rmsnorm(e->x, e->partial, split, stride, L.ffn_norm, c.weight_dtype, c.rms_eps, T, d, e->act_norm, ad,
                           e->stream, e->stamp(K_OTHER), f8 ? e->a8_norm.data : nullptr, e->a8_norm.rows,
                           f8 ? e->a8_norm.scale : nullptr, &e->norm_split);
    e->count(n, K_OTHER);
    int s_gu;
    if (c.weight_dtype == SLED_BF16 && linear_split(e, T, L.gate_up) == 1) {
      // the whole sum is formed in one place: SwiGLU is applied there, act_ffn comes straight out of the GEMM
      TcEpilogue epi;
      epi.mode = kEpiSwiglu;
      epi.act_out = static_cast<__nv_bfloat16*>(e->act_ffn);
      epi.act_ld = c.ffn_dim;
      rc = run_linear(e, e->act_norm, &e->tc_norm, L.gate_up, T, nullptr, &s_gu, epi);
      if (rc) return rc;
    } else {
      rc = run_linear(e, e->act_norm, &e->tc_norm, L.gate_up, T, nullptr, &s_gu);
      if (rc) return rc;
      e->mark(K_OTHER);
      n = launch_swiglu(e->partial, s_gu, static_cast<int64_t>(T) * L.gate_up.N, T, c.ffn_dim, e->act_ffn, ad, e->stream,
                        e->stamp(K_OTHER));
      e->count(n, K_OTHER);
    }
    rc = run_linear(e, e->act_ffn, &e->tc_ffn, L.down, T, nullptr, &split);
    if (rc) return rc;
    stride = static_cast<int64_t>(T) * L.down.N;
  }
  if (need_logits) {
    e->mark(K_OTHER);
    n = launch_add_rmsnorm(e->x, e->partial, split, stride, e->final_norm, c.weight_dtype, c.rms_eps, T, d, e->act_norm,
                           ad, e->stream, e->stamp(K_OTHER), f8 ? e->a8_norm.data : nullptr, e->a8_norm.rows,
                           f8 ? e->a8_norm.scale : nullptr, &e->norm_split);
    e->count(n, K_OTHER);
    int s1;
    int rc = run_linear(e, e->act_norm, &e->tc_norm, e->lm_head, T, e->logits, &s1);
    if (rc) return rc;
  }
  return SLED_OK;
}

int upload_meta(sled_engine* e) {
  CU_TRY(cudaMemcpyAsync(e->d_meta, e->h_meta, align_up(e->meta_used, 16), cudaMemcpyHostToDevice, e->stream));
  return SLED_OK;
}

// Timing mode 1.  Launches overlap (a kernel may begin while its predecessor drains), so a launch is charged the
// time by which it extends the step beyond everything launched before it: end_i - max(begin_i, latest end so far);
// stretches in which nothing ran go to ms_idle.  The parts add up to ms_step = last end - first begin.
int finish_stamps(sled_engine* e) {
  const size_t n = e->stamp_used, cap = e->stamp_cap;
  if (n == 0) return SLED_OK;
  CU_TRY(cudaMemcpy(e->h_stamps, e->d_stamps, sizeof(unsigned long long) * 2 * cap, cudaMemcpyDeviceToHost));
  double acc[K_KINDS] = {0, 0, 0, 0}, idle = 0.0;
  unsigned long long first = 0, latest = 0;
  bool any = false;
  for (size_t i = 0; i < n; ++i) {
    const unsigned long long b = e->h_stamps[i], en = e->h_stamps[cap + i];
    if (en == 0 || b == ~0ull) continue;   // nothing was launched for this slot
    if (!any) { first = latest = b; any = true; }
    if (b > latest) idle += static_cast<double>(b - latest);
    const unsigned long long from = b > latest ? b : latest;
    if (en > from) acc[e->stamp_kind[i]] += static_cast<double>(en - from);
    if (en > latest) latest = en;
  }
  e->st.ms_linear = static_cast<float>(acc[K_LINEAR] * 1e-6);
  e->st.ms_attention = static_cast<float>(acc[K_ATTN] * 1e-6);
  e->st.ms_accept = static_cast<float>(acc[K_ACCEPT] * 1e-6);
  e->st.ms_other = static_cast<float>(acc[K_OTHER] * 1e-6);
  e->st.ms_idle = static_cast<float>(idle * 1e-6);
  e->st.ms_step = static_cast<float>(static_cast<double>(latest - first) * 1e-6);
  return SLED_OK;
}

int finish_timing(sled_engine* e) {
  if (e->timing == 1) return finish_stamps(e);
  e->st.ms_idle = 0.f;
  if (e->timing != 2 || e->ev_used < 2) return SLED_OK;
  float acc[K_KINDS] = {0, 0, 0, 0};
  for (size_t i = 0; i + 1 < e->ev_used; ++i) {
    float ms = 0.f;
    CU_TRY(cudaEventElapsedTime(&ms, e->ev_pool[i], e->ev_pool[i + 1]));
    acc[e->ev_kind[i]] += ms;
  }
  float total = 0.f;
  CU_TRY(cudaEventElapsedTime(&total, e->ev_pool[0], e->ev_pool[e->ev_used - 1]));
  e->st.ms_linear = acc[K_LINEAR];
  e->st.ms_attention = acc[K_ATTN];
  e->st.ms_accept = acc[K_ACCEPT];
  e->st.ms_other = acc[K_OTHER];
  e->st.ms_step = total;
  return SLED_OK;
}

int check_tc_error(sled_engine* e) {
  if (!e->tc_error) return SLED_OK;
  int32_t v = 0;
  CU_TRY(cudaMemcpy(&v, e->tc_error, sizeof(v), cudaMemcpyDeviceToHost));
  if (v != 0) {
    std::fprintf(stderr, "sled: a kernel gave up waiting (code %d)\n", v);
    cudaMemset(e->tc_error, 0, sizeof(v));
    return SLED_ERR_DEVICE;
  }
  return SLED_OK;
}

void begin_step(sled_engine* e) {
  e->meta_used = 0;
  e->ev_used = 0;
  e->stamp_used = 0;
  if (e->timing == 1) {   // begin words to all ones (a minimum is taken), end words to zero (a maximum)
    cudaMemsetAsync(e->d_stamps, 0xFF, sizeof(unsigned long long) * e->stamp_cap, e->stream);
    cudaMemsetAsync(e->d_stamps + e->stamp_cap, 0, sizeof(unsigned long long) * e->stamp_cap, e->stream);
  }
  e->launches_step = 0;
  e->lin_launches = 0;
  e->attn_launches = 0;
}

void destroy(sled_engine* e) {
  if (!e) return;
  cudaSetDevice(e->cfg.device_index);
  if (e->stream) cudaStreamSynchronize(e->stream);
  for (auto& L : e->layers) {
    tc_weight_free(&L.qkv.tc); tc_weight_free(&L.o.tc); tc_weight_free(&L.gate_up.tc); tc_weight_free(&L.down.tc);
  }
  tc_weight_free(&e->lm_head.tc);
  for (void* p : e->allocs) cudaFree(p);
  if (e->h_meta) cudaFreeHost(e->h_meta);
  if (e->h_results) cudaFreeHost(e->h_results);
  if (e->h_stamps) cudaFreeHost(e->h_stamps);
  for (auto ev : e->ev_pool) cudaEventDestroy(ev);
  if (e->ev_copy) cudaEventDestroy(e->ev_copy);
  if (e->ev_a) cudaEventDestroy(e->ev_a);
  if (e->ev_b) cudaEventDestroy(e->ev_b);
  if (e->copy_stream) cudaStreamDestroy(e->copy_stream);
  if (e->own_stream && e->stream) cudaStreamDestroy(e->stream);
  delete e->kvm;
  delete e->planner;
  delete e;
}

// copies src (host or device) into a fresh device allocation
int upload(sled_engine* e, const void* src, size_t bytes, void** dst) {
  if (!src) return SLED_ERR_ARG;
  int rc = dmalloc(e, dst, bytes);
  if (rc) return rc;
  CU_TRY(cudaMemcpy(*dst, src, bytes, cudaMemcpyDefault));
  return SLED_OK;
}

// bf16 weights: replaces the row-major matrix `rowmajor` (a plain cudaMalloc that this call frees) by its tiled copy
// 8- and 4-bit weights share everything but the weight operand's storage (w8: either of them)
bool w8(const sled_engine* e) { return e->cfg.linear_weight_bits == 8 || e->cfg.linear_weight_bits == 4; }
bool w4(const sled_engine* e) { return e->cfg.linear_weight_bits == 4; }
// bytes of one row of K weights as the caller stores them
size_t weight_row_bytes(const sled_engine* e, int K) {
  return w4(e) ? static_cast<size_t>(K) / 2 : w8(e) ? static_cast<size_t>(K) : static_cast<size_t>(K) * dtype_size(e->cfg.weight_dtype);
}

// takes over `rowmajor` (device, cudaMalloc'ed) and, for 8-bit weights, `scale` (device, [N], kept)
int finish_linear(sled_engine* e, Linear* L, void* rowmajor, float* scale, int N, int K) {
  L->N = N;
  L->K = K;
  if (w8(e)) {
    L->scale = scale;
    e->allocs.push_back(scale);
    int rc = dmalloc(e, &L->w, w4(e) ? tc_weight_f4_tiled_bytes(N, K) : tc_weight_f8_tiled_bytes(N, K));
    if (!rc && (w4(e) ? tc_weight_init_f4(&L->tc, rowmajor, L->w, scale, N, K)
                      : tc_weight_init_f8(&L->tc, rowmajor, L->w, scale, N, K)) != 0)
      rc = SLED_ERR_ARG;
    cudaFree(rowmajor);
    return rc;
  }
  if (e->cfg.weight_dtype != SLED_BF16) {
    L->w = rowmajor;
    e->allocs.push_back(rowmajor);
    return SLED_OK;
  }
  int rc = dmalloc(e, &L->w, tc_weight_tiled_bytes(N, K));
  if (!rc && tc_weight_init(&L->tc, rowmajor, L->w, N, K) != 0) rc = SLED_ERR_ARG;
  cudaFree(rowmajor);
  return rc;
}

struct Part { const void* w; const float* scale; int rows; };

int make_linear(sled_engine* e, Linear* L, std::initializer_list<Part> parts, int K) {
  // concatenates the row blocks of `parts` (and, for 8-bit weights, their scales) into one [N][K] matrix
  const size_t row_bytes = weight_row_bytes(e, K);
  int N = 0;
  for (auto& p : parts) {
    if (!p.w || (w8(e) && !p.scale)) return SLED_ERR_ARG;
    N += p.rows;
  }
  void* tmp = nullptr;
  float* scale = nullptr;
  CU_TRY(cudaMalloc(&tmp, static_cast<size_t>(N) * row_bytes));
  if (w8(e) && cudaMalloc(reinterpret_cast<void**>(&scale), sizeof(float) * N) != cudaSuccess) {
    cudaFree(tmp);
    return SLED_ERR_DEVICE;
  }
  size_t off = 0, row = 0;
  for (auto& p : parts) {
    const size_t bytes = static_cast<size_t>(p.rows) * row_bytes;
    if (cudaMemcpy(static_cast<char*>(tmp) + off, p.w, bytes, cudaMemcpyDefault) != cudaSuccess ||
        (scale && cudaMemcpy(scale + row, p.scale, sizeof(float) * p.rows, cudaMemcpyDefault) != cudaSuccess)) {
      cudaFree(tmp);
      if (scale) cudaFree(scale);
      return SLED_ERR_DEVICE;
    }
    off += bytes;
    row += p.rows;
  }
  return finish_linear(e, L, tmp, scale, N, K);
}

// gate and up projections as one matrix with their rows interleaved (row 2f = gate f, row 2f+1 = up f),
// so that a pair sits in neighbouring rows of an output tile and SwiGLU can be applied where the sums end up
int make_gate_up(sled_engine* e, Linear* L, const Part& gate, const Part& up, int F, int K) {
  if (!gate.w || !up.w || (w8(e) && (!gate.scale || !up.scale))) return SLED_ERR_ARG;
  const size_t row = weight_row_bytes(e, K);
  void* tmp = nullptr;
  float* scale = nullptr;
  CU_TRY(cudaMalloc(&tmp, 2 * static_cast<size_t>(F) * row));
  bool bad = cudaMemcpy2D(tmp, 2 * row, gate.w, row, row, F, cudaMemcpyDefault) != cudaSuccess ||
             cudaMemcpy2D(static_cast<char*>(tmp) + row, 2 * row, up.w, row, row, F, cudaMemcpyDefault) != cudaSuccess;
  if (!bad && w8(e)) {
    bad = cudaMalloc(reinterpret_cast<void**>(&scale), sizeof(float) * 2 * F) != cudaSuccess ||
          cudaMemcpy2D(scale, 2 * sizeof(float), gate.scale, sizeof(float), sizeof(float), F, cudaMemcpyDefault) != cudaSuccess ||
          cudaMemcpy2D(scale + 1, 2 * sizeof(float), up.scale, sizeof(float), sizeof(float), F, cudaMemcpyDefault) != cudaSuccess;
  }
  if (bad) {
    cudaFree(tmp);
    if (scale) cudaFree(scale);
    return SLED_ERR_DEVICE;
  }
  return finish_linear(e, L, tmp, scale, 2 * F, K);
}

int check_cfg(const sled_config& c) {
  if (c.n_layers <= 0 || c.d_model <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.head_dim <= 0 || c.ffn_dim <= 0 ||
      c.vocab <= 0)
    return SLED_ERR_ARG;
  if (c.n_q_heads % c.n_kv_heads) return SLED_ERR_ARG;
  if (c.head_dim != 32 && c.head_dim != 64 && c.head_dim != 128) return SLED_ERR_ARG;
  if (c.d_model % 8 || c.ffn_dim % 8) return SLED_ERR_ARG;
  if (c.weight_dtype != SLED_F32 && c.weight_dtype != SLED_BF16) return SLED_ERR_ARG;
  if (c.kv_dtype != SLED_F32 && c.kv_dtype != SLED_BF16) return SLED_ERR_ARG;
  if (c.weight_dtype == SLED_BF16 && c.kv_dtype != SLED_BF16) return SLED_ERR_ARG;
  if (c.draft_probs_dtype != SLED_F32 && c.draft_probs_dtype != SLED_BF16) return SLED_ERR_ARG;
  if (c.attention_impl != 0 && c.attention_impl != 1) return SLED_ERR_ARG;
  const bool narrow = c.linear_weight_bits == 8 || c.linear_weight_bits == 4;
  if (c.linear_weight_bits != 0 && c.linear_weight_bits != 16 && !narrow) return SLED_ERR_ARG;
  if (narrow && c.weight_dtype != SLED_BF16) return SLED_ERR_ARG;
  if (narrow && (c.d_model % 16 || c.ffn_dim % 16 || (c.n_q_heads * c.head_dim) % 16)) return SLED_ERR_ARG;
  if (c.page_size <= 0 || c.n_pages <= 0 || c.max_batch <= 0 || c.max_k < 0 || c.max_step_tokens <= 0)
    return SLED_ERR_ARG;
  if (c.max_step_tokens < c.max_k + 1) return SLED_ERR_ARG;
  if (!(c.temperature > 0.f) || !(c.rms_eps > 0.f) || !(c.rope_theta > 0.f)) return SLED_ERR_ARG;
  return SLED_OK;
}

}  // namespace

// =================================================================== C boundary ==
extern "C" {

const char* sled_strerror(int s) {
  switch (s) {
    case SLED_OK: return "ok";
    case SLED_ERR_ARG: return "bad argument";
    case SLED_ERR_UNKNOWN_CTX: return "unknown context";
    case SLED_ERR_DUP_CTX: return "duplicate context";
    case SLED_ERR_K_RANGE: return "draft count out of range";
    case SLED_ERR_TOKEN_RANGE: return "token id out of range";
    case SLED_ERR_NO_PAGES: return "KV pool exhausted";
    case SLED_ERR_BATCH_TOO_LARGE: return "batch too large";
    case SLED_ERR_NONFINITE: return "non-finite logit";
    case SLED_ERR_DEVICE: return "device error";
    case SLED_ERR_NO_DEVICE: return "no CUDA device (this library has no CPU fallback)";
    case SLED_ERR_BASE_LEN: return "base_len outside the context's known history";
    default: return "unknown status";
  }
}

int sled_init(const sled_weights* w, const sled_config* cfg, sled_engine** out) {
  if (!w || !cfg || !out) return SLED_ERR_ARG;
  *out = nullptr;
  int rc = check_cfg(*cfg);
  if (rc) return rc;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) {
    cudaGetLastError();
    return SLED_ERR_NO_DEVICE;
  }
  if (cfg->device_index < 0 || cfg->device_index >= n_dev) return SLED_ERR_ARG;
  if (cudaSetDevice(cfg->device_index) != cudaSuccess) return SLED_ERR_NO_DEVICE;
  sled_engine* e = new (std::nothrow) sled_engine();
  if (!e) return SLED_ERR_DEVICE;
  e->cfg = *cfg;
  const sled_config& c = e->cfg;
  auto fail = [&](int code) { destroy(e); return code; };
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, c.device_index) != cudaSuccess) return fail(SLED_ERR_NO_DEVICE);
  e->n_sm = prop.multiProcessorCount;
  if (c.weight_dtype == SLED_BF16 && prop.major != 10) {
    std::fprintf(stderr, "sled: the bf16 path needs an sm_100 device (found sm_%d%d)\n", prop.major, prop.minor);
    return fail(SLED_ERR_NO_DEVICE);
  }
  if (c.stream) e->stream = static_cast<cudaStream_t>(c.stream);
  else {
    if (cudaStreamCreateWithFlags(&e->stream, cudaStreamNonBlocking) != cudaSuccess) return fail(SLED_ERR_DEVICE);
    e->own_stream = true;
  }
  if (cudaStreamCreateWithFlags(&e->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if (cudaEventCreateWithFlags(&e->ev_copy, cudaEventDisableTiming) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if (cudaEventCreate(&e->ev_a) != cudaSuccess || cudaEventCreate(&e->ev_b) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  e->kvm = new KvManager(c.n_pages, c.page_size);
  e->planner = new Planner(kBatchContinuous, 0, c.max_batch, c.max_step_tokens);

  const size_t es = dtype_size(c.weight_dtype);
  const int d = c.d_model, qd = c.n_q_heads * c.head_dim, kd = c.n_kv_heads * c.head_dim, F = c.ffn_dim;
  if ((rc = upload(e, w->tok_emb, static_cast<size_t>(c.vocab) * d * es, &e->tok_emb))) return fail(rc);
  if ((rc = upload(e, w->final_norm, d * es, &e->final_norm))) return fail(rc);
  const bool q8 = c.linear_weight_bits == 8 || c.linear_weight_bits == 4;
  if (q8 && (!w->wq_scale || !w->wk_scale || !w->wv_scale || !w->wo_scale || !w->w_gate_scale || !w->w_up_scale ||
             !w->w_down_scale))
    return fail(SLED_ERR_ARG);
  auto sc = [&](const float* const* arr, int l) { return q8 ? arr[l] : nullptr; };
  if ((rc = make_linear(e, &e->lm_head, {{w->lm_head, q8 ? w->lm_head_scale : nullptr, c.vocab}}, d))) return fail(rc);
  if (!w->attn_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->ffn_norm || !w->w_gate || !w->w_up || !w->w_down)
    return fail(SLED_ERR_ARG);
  e->layers.resize(c.n_layers);
  for (int l = 0; l < c.n_layers; ++l) {
    Layer& L = e->layers[l];
    if ((rc = upload(e, w->attn_norm[l], d * es, &L.attn_norm))) return fail(rc);
    if ((rc = upload(e, w->ffn_norm[l], d * es, &L.ffn_norm))) return fail(rc);
    if ((rc = make_linear(e, &L.qkv, {{w->wq[l], sc(w->wq_scale, l), qd}, {w->wk[l], sc(w->wk_scale, l), kd},
                                      {w->wv[l], sc(w->wv_scale, l), kd}}, d)))
      return fail(rc);
    if ((rc = make_linear(e, &L.o, {{w->wo[l], sc(w->wo_scale, l), d}}, qd))) return fail(rc);
    if ((rc = make_gate_up(e, &L.gate_up, {w->w_gate[l], sc(w->w_gate_scale, l), F}, {w->w_up[l], sc(w->w_up_scale, l), F}, F, d)))
      return fail(rc);
    if ((rc = make_linear(e, &L.down, {{w->w_down[l], sc(w->w_down_scale, l), d}}, F))) return fail(rc);
  }

  // KV pool: per layer [page][Hkv][page_size][h]
  e->kv_layer_bytes = static_cast<size_t>(c.n_pages) * c.n_kv_heads * c.page_size * c.head_dim * dtype_size(c.kv_dtype);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->kpool), e->kv_layer_bytes * c.n_layers))) return fail(rc);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->vpool), e->kv_layer_bytes * c.n_layers))) return fail(rc);

  if ((cudaMemset(e->kpool, 0, e->kv_layer_bytes * c.n_layers)) != cudaSuccess) return fail(SLED_ERR_DEVICE);  // never-written slots are read (and masked): keep them finite
  if ((cudaMemset(e->vpool, 0, e->kv_layer_bytes * c.n_layers)) != cudaSuccess) return fail(SLED_ERR_DEVICE);

  // step workspaces
  const size_t maxT = c.max_step_tokens, as = dtype_size(e->adtype());
  const size_t padT = align_up(maxT, 256);  // activation buffers are read in row tiles by the tensor-core path
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->x), maxT * d * 4))) return fail(rc);
  if ((rc = dmalloc(e, &e->act_norm, padT * d * as))) return fail(rc);
  if ((rc = dmalloc(e, &e->q_buf, maxT * qd * as))) return fail(rc);
  if ((rc = dmalloc(e, &e->attn_out, padT * qd * as))) return fail(rc);
  if ((rc = dmalloc(e, &e->act_ffn, padT * F * as))) return fail(rc);
  if ((cudaMemset(e->act_norm, 0, padT * d * as)) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if ((cudaMemset(e->attn_out, 0, padT * qd * as)) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if ((cudaMemset(e->act_ffn, 0, padT * F * as)) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->logits), maxT * c.vocab * 4))) return fail(rc);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->rope_cs), maxT * (c.head_dim / 2) * sizeof(float2)))) return fail(rc);
  {
    size_t need = 0;
    const Linear* shapes[4] = {&e->layers[0].qkv, &e->layers[0].o, &e->layers[0].gate_up, &e->layers[0].down};
    for (const Linear* L : shapes)
      for (int T = 1; T <= static_cast<int>(maxT); ++T)
        need = std::max(need, static_cast<size_t>(linear_split(e, T, *L)) * T * L->N);
    e->partial_elems = need;
    if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->partial), need * 4))) return fail(rc);
  }
  e->part_rows_cap = 8192;
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->part_acc), static_cast<size_t>(e->part_rows_cap) * qd * 4))) return fail(rc);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->part_ml), static_cast<size_t>(e->part_rows_cap) * c.n_q_heads * 8))) return fail(rc);
  if (!c.probs_on_device && !c.greedy)
    if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->q_stage), maxT * c.vocab * dtype_size(c.draft_probs_dtype)))) return fail(rc);
  // results block: [0] error word (+3 words of padding), then 3 words per request
  if (cudaMallocHost(reinterpret_cast<void**>(&e->h_results), sizeof(int32_t) * (kResultsHead + 3 * c.max_batch)) != cudaSuccess)
    return fail(SLED_ERR_DEVICE);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->d_results), sizeof(int32_t) * (kResultsHead + 3 * c.max_batch)))) return fail(rc);
  if ((cudaMemset(e->d_results, 0, sizeof(int32_t) * kResultsHead)) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if (c.weight_dtype == SLED_BF16) {
    e->tc_error = e->d_results;
    if (c.page_size == 16 && (c.head_dim == 64 || c.head_dim == 128)) {
      e->kv_maps.resize(2 * c.n_layers);
      const long long rows = static_cast<long long>(c.n_pages) * c.n_kv_heads * c.page_size;
      for (int l = 0; l < c.n_layers; ++l)
        if (tma_map_bf16_rows(&e->kv_maps[2 * l], e->kpool + e->kv_layer_bytes * l, rows, c.head_dim, 16) ||
            tma_map_bf16_rows(&e->kv_maps[2 * l + 1], e->vpool + e->kv_layer_bytes * l, rows, c.head_dim, 16))
          return fail(SLED_ERR_DEVICE);
      e->attn_tc = c.head_dim == 128 && c.attention_impl == 1;
    }
    if (tc_activation_init(&e->tc_norm, e->act_norm, static_cast<int>(padT), d) ||
        tc_activation_init(&e->tc_attn, e->attn_out, static_cast<int>(padT), qd) ||
        tc_activation_init(&e->tc_ffn, e->act_ffn, static_cast<int>(padT), F))
      return fail(SLED_ERR_DEVICE);
    if (q8) {
      struct { TcActivation8* a; int K; } parts[3] = {{&e->a8_norm, d}, {&e->a8_attn, qd}, {&e->a8_ffn, F}};
      for (auto& p : parts) {
        void* data = nullptr;
        float* sc = nullptr;
        if ((rc = dmalloc(e, &data, 2 * padT * p.K)) || (rc = dmalloc(e, reinterpret_cast<void**>(&sc), padT * sizeof(float))))
          return fail(rc);
        if (cudaMemset(data, 0, 2 * padT * p.K) != cudaSuccess || cudaMemset(sc, 0, padT * sizeof(float)) != cudaSuccess ||
            tc_activation8_init(p.a, data, sc, static_cast<int>(padT), p.K))
          return fail(SLED_ERR_DEVICE);
      }
    }
  }

  // metadata staging: tokens, requests, page table (every page at most once, plus one partial page per request), items
  const size_t max_items = static_cast<size_t>(c.n_kv_heads) * (static_cast<size_t>(c.n_pages) * c.page_size / 256 + c.max_batch + 1);
  e->meta_cap = 5 * maxT * 4 + 7 * (c.max_batch + 1) * 4 + 64 + (static_cast<size_t>(c.n_pages) + c.max_batch) * 4 +
                max_items * sizeof(int4) + 6 * c.max_batch * 8 + 64 * 16;
  if (cudaMallocHost(reinterpret_cast<void**>(&e->h_meta), e->meta_cap) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  if ((rc = dmalloc(e, reinterpret_cast<void**>(&e->d_meta), e->meta_cap))) return fail(rc);
  if ((cudaDeviceSynchronize()) != cudaSuccess) return fail(SLED_ERR_DEVICE);
  e->st.pages_total = c.n_pages;
  *out = e;
  return SLED_OK;
}

void sled_shutdown(sled_engine* e) { destroy(e); }

void* sled_get_stream(sled_engine* e) { return e ? e->stream : nullptr; }

int sled_set_sampling(sled_engine* e, float temperature, int32_t greedy) {
  if (!e || !(temperature > 0.f)) return SLED_ERR_ARG;
  if (!greedy && !e->cfg.probs_on_device && !e->q_stage) {
    cudaSetDevice(e->cfg.device_index);
    int rc = dmalloc(e, reinterpret_cast<void**>(&e->q_stage),
                     static_cast<size_t>(e->cfg.max_step_tokens) * e->cfg.vocab * dtype_size(e->cfg.draft_probs_dtype));
    if (rc) return rc;
  }
  e->cfg.temperature = temperature;
  e->cfg.greedy = greedy ? 1 : 0;
  return SLED_OK;
}

int sled_get_stats(sled_engine* e, sled_stats* out) {
  if (!e || !out) return SLED_ERR_ARG;
  e->st.pages_free = e->kvm->free_pages();
  e->st.contexts_open = e->kvm->open_contexts();
  *out = e->st;
  return SLED_OK;
}

int sled_release(sled_engine* e, uint64_t ctx_id) {
  if (!e) return SLED_ERR_ARG;
  return e->kvm->release(ctx_id);
}

int sled_prefill(sled_engine* e, uint64_t ctx_id, const int32_t* tokens, int32_t n) {
  if (!e || !tokens || n < 1) return SLED_ERR_ARG;
  for (int i = 0; i < n; ++i)
    if (tokens[i] < 0 || tokens[i] >= e->cfg.vocab) return SLED_ERR_TOKEN_RANGE;
  if (e->kvm->find(ctx_id)) return SLED_ERR_DUP_CTX;
  const int64_t need_pages = (static_cast<int64_t>(n) - 1 + e->cfg.page_size - 1) / e->cfg.page_size;
  if (need_pages > e->kvm->free_pages()) return SLED_ERR_NO_PAGES;
  cudaSetDevice(e->cfg.device_index);
  int rc = e->kvm->open(ctx_id, 0, tokens[0]);
  if (rc) return rc;
  int done = 0;
  const int n_kv = n - 1;
  while (done < n_kv) {
    const int chunk = std::min(n_kv - done, e->cfg.max_step_tokens);
    int32_t extra = chunk;
    rc = e->kvm->reserve_batch(&ctx_id, &extra, 1);
    if (!rc) {
      begin_step(e);
      std::vector<PlanReq> plan{{ctx_id, tokens + done, chunk}};
      Packed pk;
      rc = pack_step(e, plan, false, &pk);
      if (!rc) rc = upload_meta(e);
      if (!rc) rc = run_forward(e, pk, false);
      if (!rc && cudaStreamSynchronize(e->stream) != cudaSuccess) rc = SLED_ERR_DEVICE;
      if (!rc) rc = check_tc_error(e);
      e->st.kernels_launched += e->launches_step;
    }
    if (rc) {
      e->kvm->release(ctx_id);
      return rc;
    }
    e->kvm->commit(ctx_id, chunk, tokens[done + chunk], tokens + done + 1);
    done += chunk;
  }
  e->kvm->truncate(ctx_id, n_kv, tokens[n - 1]);
  return SLED_OK;
}

int sled_verify_batch(sled_engine* e, const sled_request* reqs, int32_t n_reqs, uint64_t seed, sled_result* results) {
  if (!e || n_reqs < 0 || (n_reqs > 0 && (!reqs || !results))) return SLED_ERR_ARG;
  if (n_reqs == 0) return SLED_OK;
  const sled_config& c = e->cfg;
  if (n_reqs > c.max_batch) return SLED_ERR_BATCH_TOO_LARGE;
  // ---- validation: nothing is changed before every request has passed
  int64_t T = 0;
  for (int i = 0; i < n_reqs; ++i) {
    const sled_request& r = reqs[i];
    if (r.k < 0 || r.k > c.max_k) return SLED_ERR_K_RANGE;
    if (r.k > 0 && !r.draft_tokens) return SLED_ERR_ARG;
    if (r.k > 0 && !c.greedy && !r.draft_probs) return SLED_ERR_ARG;
    if (r.base_len < 0) return SLED_ERR_ARG;
    for (int j = 0; j < r.k; ++j)
      if (r.draft_tokens[j] < 0 || r.draft_tokens[j] >= c.vocab) return SLED_ERR_TOKEN_RANGE;
    T += r.k + 1;
  }
  if (T > c.max_step_tokens) return SLED_ERR_BATCH_TOO_LARGE;
  std::vector<uint64_t> ctxs(n_reqs);
  std::vector<int32_t> extra(n_reqs);
  std::vector<int64_t> base(n_reqs);
  for (int i = 0; i < n_reqs; ++i) { ctxs[i] = reqs[i].ctx_id; extra[i] = reqs[i].k + 1; base[i] = reqs[i].base_len; }
  // unknown / duplicate context, base_len out of range, no pages: nothing has changed.  Otherwise contexts whose
  // request names a base_len are cut back to it here, and stay there whatever happens later in the call.
  int rc = e->kvm->reserve_batch(ctxs.data(), extra.data(), n_reqs, base.data());
  if (rc) return rc;
  std::vector<int32_t> old_pending(n_reqs);
  for (int i = 0; i < n_reqs; ++i) old_pending[i] = e->kvm->find(ctxs[i])->pending;
  bool issued = false;   // device work of this call is queued (copies or kernels)
  auto rollback = [&](int code) {
    if (issued) {        // nothing may still read the staging buffers or write the pages that go back to the pool
      cudaStreamSynchronize(e->copy_stream);
      cudaStreamSynchronize(e->stream);
      cudaGetLastError();
    }
    for (int i = 0; i < n_reqs; ++i) e->kvm->commit(ctxs[i], 0, old_pending[i]);
    return code;
  };
  if (cudaSetDevice(c.device_index) != cudaSuccess) return rollback(SLED_ERR_DEVICE);

  // ---- pack
  begin_step(e);
  std::vector<int32_t> fed(T);
  std::vector<PlanReq> plan(n_reqs);
  {
    int t = 0;
    for (int i = 0; i < n_reqs; ++i) {
      plan[i] = {ctxs[i], fed.data() + t, reqs[i].k + 1};
      fed[t++] = old_pending[i];
      for (int j = 0; j < reqs[i].k; ++j) fed[t++] = reqs[i].draft_tokens[j];
    }
  }
  Packed pk;
  if ((rc = pack_step(e, plan, false, &pk))) return rollback(rc);
  uint32_t *d_lo = nullptr, *d_hi = nullptr;
  const void** d_qptr = nullptr;
  uint32_t* h_lo = e->meta_alloc<uint32_t>(n_reqs, &d_lo);
  uint32_t* h_hi = e->meta_alloc<uint32_t>(n_reqs, &d_hi);
  const void** h_qptr = e->meta_alloc<const void*>(n_reqs, &d_qptr);
  if (!h_lo || !h_hi || !h_qptr) return rollback(SLED_ERR_BATCH_TOO_LARGE);
  bool staged = false;
  struct QCopy { char* dst; const void* src; size_t bytes; };
  const size_t qsize = dtype_size(c.draft_probs_dtype);
  std::vector<QCopy> copies;
  {
    size_t row = 0;
    for (int i = 0; i < n_reqs; ++i) {
      h_lo[i] = static_cast<uint32_t>(ctxs[i]);
      h_hi[i] = static_cast<uint32_t>(ctxs[i] >> 32);
      h_qptr[i] = nullptr;
      if (reqs[i].k > 0 && !c.greedy) {
        cudaPointerAttributes attr{};
        const bool on_device = cudaPointerGetAttributes(&attr, reqs[i].draft_probs) == cudaSuccess &&
                               attr.type == cudaMemoryTypeDevice;
        cudaGetLastError();
        if (on_device && attr.device != c.device_index) return rollback(SLED_ERR_ARG);   // another GPU's memory
        if (on_device) h_qptr[i] = reqs[i].draft_probs;   // read in place by the acceptance kernel
        else if (!e->q_stage) return rollback(SLED_ERR_ARG);  // engine was created for device-resident rows only
        else {
          // draft distributions travel on the copy stream while the forward pass runs
          char* dst = reinterpret_cast<char*>(e->q_stage) + row * c.vocab * qsize;
          copies.push_back({dst, reqs[i].draft_probs, static_cast<size_t>(reqs[i].k) * c.vocab * qsize});
          h_qptr[i] = dst;
          row += reqs[i].k;
          staged = true;
        }
      }
    }
  }
  // the step's description goes first: the forward pass waits for it, the draft rows are not needed before the
  // acceptance kernel (copies in one direction are served in the order they were issued)
  issued = true;
  if ((rc = upload_meta(e))) return rollback(rc);
  for (const QCopy& qc : copies)
    if (cudaMemcpyAsync(qc.dst, qc.src, qc.bytes, cudaMemcpyHostToDevice, e->copy_stream) != cudaSuccess)
      return rollback(SLED_ERR_DEVICE);
  if (staged && cudaEventRecord(e->ev_copy, e->copy_stream) != cudaSuccess) return rollback(SLED_ERR_DEVICE);

  // ---- forward + acceptance
  if (e->probe_wait_cycles > 0) {   // self-test armed by sled_debug_arm_wait_timeout: this step will be reported as failed
    const int n_probe = tc_wait_probe_launch(e->tc_error, e->probe_wait_cycles, e->stream);
    e->probe_wait_cycles = 0;
    if (n_probe < 0) return rollback(SLED_ERR_DEVICE);
    e->count(n_probe, K_OTHER);
  }
  if ((rc = run_forward(e, pk, true))) return rollback(rc);
  if (staged && cudaStreamWaitEvent(e->stream, e->ev_copy, 0) != cudaSuccess) return rollback(SLED_ERR_DEVICE);
  AcceptArgs aa{};
  aa.logits = e->logits;
  aa.cu_q = pk.cu_q;
  aa.ids = pk.ids;
  aa.q_rows = c.greedy ? nullptr : d_qptr;
  aa.q_bf16 = c.draft_probs_dtype == SLED_BF16;
  aa.ctx_lo = d_lo;
  aa.ctx_hi = d_hi;
  aa.pos0 = pk.kv_base;
  aa.results = e->d_results + kResultsHead;
  aa.B = n_reqs;
  aa.V = c.vocab;
  aa.inv_tau = 1.0f / c.temperature;
  aa.greedy = c.greedy;
  aa.seed = seed;
  e->mark(K_ACCEPT);
  aa.stamp = e->stamp(K_ACCEPT);
  int n = launch_accept(aa, e->stream);
  if (n < 0) return rollback(SLED_ERR_DEVICE);
  e->count(n, K_ACCEPT);
  e->mark(K_OTHER);
  cudaError_t err = cudaMemcpyAsync(e->h_results, e->d_results, sizeof(int32_t) * (kResultsHead + 3 * n_reqs),
                                    cudaMemcpyDeviceToHost, e->stream);
  if (err == cudaSuccess) err = cudaStreamSynchronize(e->stream);
  if (err == cudaSuccess) err = cudaGetLastError();
  if (err != cudaSuccess) {
    std::fprintf(stderr, "sled: verification step failed on the device: %s\n", cudaGetErrorString(err));
    return rollback(SLED_ERR_DEVICE);
  }
  if (e->h_results[0] != 0) {   // a bounded device-side wait ran out somewhere in the step: nothing of it is kept
    std::fprintf(stderr, "sled: a kernel of the step gave up waiting (code %d)\n", e->h_results[0]);
    cudaMemsetAsync(e->d_results, 0, sizeof(int32_t), e->stream);
    cudaStreamSynchronize(e->stream);
    return rollback(SLED_ERR_DEVICE);
  }
  e->last_T = pk.T;
  finish_timing(e);

  // ---- feedback, then commit the accepted prefix / roll back the rest
  e->st.steps += 1;
  e->st.requests += n_reqs;
  e->st.tokens_scored += T;
  e->st.kernels_launched += e->launches_step;
  e->st.kernels_last_step = e->launches_step;
  e->st.linear_launches_last_step = e->lin_launches;
  e->st.attention_launches_last_step = e->attn_launches;
  for (int i = 0; i < n_reqs; ++i) {
    const int32_t* r = e->h_results + kResultsHead + 3 * i;
    results[i].n_accepted = r[0];
    results[i].next_token = r[1];
    results[i].status = r[2];
    if (results[i].status == SLED_OK && e->commit) {
      e->kvm->commit(ctxs[i], results[i].n_accepted + 1, results[i].next_token, reqs[i].draft_tokens);
      e->st.drafts_accepted += results[i].n_accepted;
      e->st.tokens_committed += results[i].n_accepted + 1;
    } else {
      e->kvm->commit(ctxs[i], 0, old_pending[i]);
    }
  }
  return SLED_OK;
}

// ------------------------------------------------------------------- server loop --
int sled_server_config(sled_engine* e, int32_t policy, int32_t batch_size) {
  if (!e) return SLED_ERR_ARG;
  if (!e->waiting.empty()) return SLED_ERR_ARG;   // the policy changes only while nothing is queued
  Planner* p = new Planner(policy, batch_size, e->cfg.max_batch, e->cfg.max_step_tokens);
  if (!p->valid()) {
    delete p;
    return SLED_ERR_ARG;
  }
  delete e->planner;
  e->planner = p;
  return SLED_OK;
}

int sled_submit(sled_engine* e, const sled_request* req, uint64_t* ticket) {
  if (!e || !req || !ticket) return SLED_ERR_ARG;
  const sled_config& c = e->cfg;
  if (req->k < 0 || req->k > c.max_k) return SLED_ERR_K_RANGE;
  if (req->k > 0 && (!req->draft_tokens || (!c.greedy && !req->draft_probs))) return SLED_ERR_ARG;
  if (req->base_len < 0) return SLED_ERR_ARG;
  for (int j = 0; j < req->k; ++j)
    if (req->draft_tokens[j] < 0 || req->draft_tokens[j] >= c.vocab) return SLED_ERR_TOKEN_RANGE;
  if (!e->kvm->find(req->ctx_id)) return SLED_ERR_UNKNOWN_CTX;
  const uint64_t t = e->next_ticket++;
  int rc = e->planner->push(t, req->ctx_id, req->k);
  if (rc) return rc;
  sled_engine::Waiting& w = e->waiting[t];
  w.req = *req;
  w.drafts.assign(req->draft_tokens, req->draft_tokens + req->k);
  *ticket = t;
  return SLED_OK;
}

int sled_step(sled_engine* e, uint64_t seed, int32_t flush, int32_t* n_verified) {
  if (!e) return SLED_ERR_ARG;
  if (n_verified) *n_verified = 0;
  const std::vector<uint64_t> batch = e->planner->next_batch(flush != 0);
  if (batch.empty()) return SLED_OK;
  // Requests were checked when they came in, but their context may have been released, or cut back, since: those
  // are answered with their own error; the rest of the batch runs.
  std::vector<sled_request> reqs;
  std::vector<uint64_t> tickets;
  for (uint64_t t : batch) {
    sled_engine::Waiting& w = e->waiting[t];
    w.req.draft_tokens = w.drafts.data();
    const CtxState* cs = e->kvm->find(w.req.ctx_id);
    int bad = SLED_OK;
    if (!cs) bad = SLED_ERR_UNKNOWN_CTX;
    else if (w.req.base_len != 0 && (w.req.base_len < cs->hist_start + 1 || w.req.base_len > cs->n_kv + 1)) bad = SLED_ERR_BASE_LEN;
    if (bad) {
      e->finished[t] = sled_result{0, -1, bad};
      e->waiting.erase(t);
      continue;
    }
    reqs.push_back(w.req);
    tickets.push_back(t);
  }
  if (reqs.empty()) return SLED_OK;
  std::vector<sled_result> res(reqs.size());
  const int rc = sled_verify_batch(e, reqs.data(), static_cast<int32_t>(reqs.size()), seed, res.data());
  for (size_t i = 0; i < tickets.size(); ++i) {
    e->finished[tickets[i]] = rc == SLED_OK ? res[i] : sled_result{0, -1, rc};   // a failed step answers every request with its code
    e->waiting.erase(tickets[i]);
  }
  if (rc == SLED_OK && n_verified) *n_verified = static_cast<int32_t>(tickets.size());
  return rc;
}

int sled_poll(sled_engine* e, uint64_t ticket, sled_result* out) {
  if (!e || !out) return SLED_ERR_ARG;
  auto it = e->finished.find(ticket);
  if (it == e->finished.end()) return e->waiting.count(ticket) ? SLED_PENDING : SLED_ERR_ARG;
  *out = it->second;
  e->finished.erase(it);
  return SLED_OK;
}

int32_t sled_queued(sled_engine* e) { return e ? e->planner->queued() : SLED_ERR_ARG; }

// ------------------------------------------------------------ stand-alone pieces --
int sled_accept_rows(const float* logits, const int32_t* cu_rows, const int32_t* drafts, const float* q_rows,
                     const uint64_t* ctx_ids, const int64_t* pos0, int32_t n_reqs, int32_t vocab, float temperature,
                     int32_t greedy, uint64_t seed, sled_result* results, void* stream, float* device_ms) {
  if (!logits || !cu_rows || !ctx_ids || !pos0 || !results || n_reqs <= 0 || vocab <= 0 || !(temperature > 0.f))
    return SLED_ERR_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) { cudaGetLastError(); return SLED_ERR_NO_DEVICE; }
  const int rows = cu_rows[n_reqs];
  if (cu_rows[0] != 0 || rows < n_reqs) return SLED_ERR_ARG;
  if (rows > n_reqs && (!drafts || (!greedy && !q_rows))) return SLED_ERR_ARG;   // draft ids are read in both modes
  for (int i = 0; i < n_reqs; ++i)
    if (cu_rows[i + 1] - cu_rows[i] < 1) return SLED_ERR_ARG;                      // checked before anything is written
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // small per-call device arrays
  std::vector<int32_t> ids(rows, 0), p0(n_reqs);
  std::vector<uint32_t> lo(n_reqs), hi(n_reqs);
  std::vector<const void*> qp(n_reqs, nullptr);
  int64_t drow = 0;
  for (int i = 0; i < n_reqs; ++i) {
    const int k = cu_rows[i + 1] - cu_rows[i] - 1;
    if (k < 0) return SLED_ERR_ARG;
    for (int j = 0; j < k; ++j) {
      const int d = drafts[drow + j];
      if (d < 0 || d >= vocab) return SLED_ERR_TOKEN_RANGE;
      ids[cu_rows[i] + 1 + j] = d;
    }
    if (q_rows && k > 0) qp[i] = q_rows + drow * vocab;
    drow += k;
    lo[i] = static_cast<uint32_t>(ctx_ids[i]);
    hi[i] = static_cast<uint32_t>(ctx_ids[i] >> 32);
    p0[i] = static_cast<int32_t>(pos0[i]);
  }
  const size_t sz_ids = align_up(rows * 4, 16), sz_b = align_up(static_cast<size_t>(n_reqs + 1) * 4, 16), sz_p = align_up(static_cast<size_t>(n_reqs) * 8, 16);
  const size_t total = sz_ids + 4 * sz_b + sz_p + align_up(static_cast<size_t>(n_reqs) * 12, 16);
  char* dev = nullptr;
  CU_TRY(cudaMalloc(reinterpret_cast<void**>(&dev), total));
  std::vector<char> host(total, 0);
  size_t off = 0;
  auto put = [&](const void* src, size_t bytes, size_t slot) { std::memcpy(host.data() + off, src, bytes); size_t o = off; off += slot; return o; };
  const size_t o_ids = put(ids.data(), rows * 4, sz_ids);
  const size_t o_cu = put(cu_rows, static_cast<size_t>(n_reqs + 1) * 4, sz_b);
  const size_t o_lo = put(lo.data(), n_reqs * 4, sz_b);
  const size_t o_hi = put(hi.data(), n_reqs * 4, sz_b);
  const size_t o_p0 = put(p0.data(), n_reqs * 4, sz_b);
  const size_t o_qp = put(qp.data(), static_cast<size_t>(n_reqs) * 8, sz_p);
  const size_t o_res = off;
  cudaError_t err = cudaMemcpyAsync(dev, host.data(), total, cudaMemcpyHostToDevice, s);
  cudaEvent_t a = nullptr, b = nullptr;
  if (err == cudaSuccess) err = cudaEventCreate(&a);
  if (err == cudaSuccess) err = cudaEventCreate(&b);
  AcceptArgs aa{};
  aa.logits = logits;
  aa.cu_q = reinterpret_cast<int32_t*>(dev + o_cu);
  aa.ids = reinterpret_cast<int32_t*>(dev + o_ids);
  aa.q_rows = greedy ? nullptr : reinterpret_cast<const void* const*>(dev + o_qp);
  aa.ctx_lo = reinterpret_cast<uint32_t*>(dev + o_lo);
  aa.ctx_hi = reinterpret_cast<uint32_t*>(dev + o_hi);
  aa.pos0 = reinterpret_cast<int32_t*>(dev + o_p0);
  aa.results = reinterpret_cast<int32_t*>(dev + o_res);
  aa.B = n_reqs;
  aa.V = vocab;
  aa.inv_tau = 1.0f / temperature;
  aa.greedy = greedy ? 1 : 0;
  aa.seed = seed;
  if (err == cudaSuccess) err = cudaEventRecord(a, s);
  int n = err == cudaSuccess ? launch_accept(aa, s) : -1;
  if (err == cudaSuccess) err = cudaEventRecord(b, s);
  std::vector<int32_t> res(static_cast<size_t>(n_reqs) * 3);
  if (err == cudaSuccess) err = cudaMemcpyAsync(res.data(), dev + o_res, res.size() * 4, cudaMemcpyDeviceToHost, s);
  if (err == cudaSuccess) err = cudaStreamSynchronize(s);
  if (err == cudaSuccess && device_ms) err = cudaEventElapsedTime(device_ms, a, b);
  if (a) cudaEventDestroy(a);
  if (b) cudaEventDestroy(b);
  cudaFree(dev);
  if (err != cudaSuccess || n < 0) {
    std::fprintf(stderr, "sled: sled_accept_rows failed: %s\n", cudaGetErrorString(err));
    return n < 0 && err == cudaSuccess ? SLED_ERR_ARG : SLED_ERR_DEVICE;
  }
  for (int i = 0; i < n_reqs; ++i) {
    results[i].n_accepted = res[3 * i];
    results[i].next_token = res[3 * i + 1];
    results[i].status = res[3 * i + 2];
  }
  return SLED_OK;
}

int sled_attention_ragged(sled_engine* e, int32_t layer, const uint64_t* ctx_ids, const int32_t* q_len, int32_t n_reqs,
                          const void* q, void* out, float* device_ms) {
  if (!e || !ctx_ids || !q_len || !q || !out || n_reqs <= 0 || layer < 0 || layer >= e->cfg.n_layers) return SLED_ERR_ARG;
  std::vector<PlanReq> plan(n_reqs);
  for (int i = 0; i < n_reqs; ++i) {
    if (q_len[i] <= 0) return SLED_ERR_ARG;
    const CtxState* c = e->kvm->find(ctx_ids[i]);
    if (!c) return SLED_ERR_UNKNOWN_CTX;
    if (c->n_kv < q_len[i]) return SLED_ERR_ARG;
    plan[i] = {ctx_ids[i], nullptr, q_len[i]};
  }
  cudaSetDevice(e->cfg.device_index);
  begin_step(e);
  Packed pk;
  int rc = pack_step(e, plan, true, &pk);
  if (rc) return rc;
  if ((rc = upload_meta(e))) return rc;
  CU_TRY(cudaEventRecord(e->ev_a, e->stream));
  int n = launch_attention(attn_args(e, pk, layer, q, out), e->stream);
  CU_TRY(cudaEventRecord(e->ev_b, e->stream));
  if (n < 0) return SLED_ERR_DEVICE;
  CU_TRY(cudaStreamSynchronize(e->stream));
  CU_TRY(cudaGetLastError());
  if ((rc = check_tc_error(e))) return rc;
  e->st.kernels_launched += n;
  if (device_ms) CU_TRY(cudaEventElapsedTime(device_ms, e->ev_a, e->ev_b));
  return SLED_OK;
}

// --------------------------------------------------------------------- hooks --
int sled_debug_load_kv(sled_engine* e, uint64_t ctx_id, const void* K, const void* V, int32_t n_tokens, int32_t pending) {
  if (!e || n_tokens < 0 || (n_tokens > 0 && (!K || !V)) || pending < 0 || pending >= e->cfg.vocab) return SLED_ERR_ARG;
  const sled_config& c = e->cfg;
  int rc = e->kvm->open(ctx_id, n_tokens, pending);
  if (rc || n_tokens == 0) return rc;
  cudaSetDevice(c.device_index);
  const CtxState* cs = e->kvm->find(ctx_id);
  std::vector<int32_t> slots(n_tokens);
  for (int i = 0; i < n_tokens; ++i) slots[i] = static_cast<int32_t>(e->kvm->slot_of(*cs, i));
  const size_t layer_bytes = static_cast<size_t>(n_tokens) * c.n_kv_heads * c.head_dim * dtype_size(c.kv_dtype);
  int32_t* d_slots = nullptr;
  char* stage = nullptr;
  auto cleanup = [&](int code) {
    cudaStreamSynchronize(e->stream);
    if (d_slots) cudaFree(d_slots);
    if (stage) cudaFree(stage);
    if (code) e->kvm->release(ctx_id);
    return code;
  };
  if (cudaMalloc(reinterpret_cast<void**>(&d_slots), slots.size() * 4) != cudaSuccess) return cleanup(SLED_ERR_DEVICE);
  if (cudaMemcpyAsync(d_slots, slots.data(), slots.size() * 4, cudaMemcpyHostToDevice, e->stream) != cudaSuccess)
    return cleanup(SLED_ERR_DEVICE);
  cudaPointerAttributes attr{};
  const bool on_device = cudaPointerGetAttributes(&attr, K) == cudaSuccess && attr.type == cudaMemoryTypeDevice;
  cudaGetLastError();
  if (!on_device && cudaMalloc(reinterpret_cast<void**>(&stage), 2 * layer_bytes) != cudaSuccess) return cleanup(SLED_ERR_DEVICE);
  for (int l = 0; l < c.n_layers; ++l) {
    const char* ksrc = static_cast<const char*>(K) + layer_bytes * l;
    const char* vsrc = static_cast<const char*>(V) + layer_bytes * l;
    if (!on_device) {
      if (cudaMemcpyAsync(stage, ksrc, layer_bytes, cudaMemcpyHostToDevice, e->stream) != cudaSuccess ||
          cudaMemcpyAsync(stage + layer_bytes, vsrc, layer_bytes, cudaMemcpyHostToDevice, e->stream) != cudaSuccess)
        return cleanup(SLED_ERR_DEVICE);
      ksrc = stage;
      vsrc = stage + layer_bytes;
    }
    launch_kv_scatter(ksrc, d_slots, n_tokens, c.n_kv_heads, c.head_dim, c.page_size, e->kpool + e->kv_layer_bytes * l, c.kv_dtype, e->stream);
    launch_kv_scatter(vsrc, d_slots, n_tokens, c.n_kv_heads, c.head_dim, c.page_size, e->vpool + e->kv_layer_bytes * l, c.kv_dtype, e->stream);
    if (!on_device && cudaStreamSynchronize(e->stream) != cudaSuccess) return cleanup(SLED_ERR_DEVICE);  // staging is reused
  }
  if (cudaStreamSynchronize(e->stream) != cudaSuccess || cudaGetLastError() != cudaSuccess) return cleanup(SLED_ERR_DEVICE);
  return cleanup(SLED_OK);
}

int sled_debug_read_kv(sled_engine* e, uint64_t ctx_id, int32_t layer, void* K, void* V, int32_t n_tokens) {
  if (!e || !K || !V || layer < 0 || layer >= e->cfg.n_layers || n_tokens <= 0) return SLED_ERR_ARG;
  const sled_config& c = e->cfg;
  const CtxState* cs = e->kvm->find(ctx_id);
  if (!cs) return SLED_ERR_UNKNOWN_CTX;
  if (n_tokens > static_cast<int64_t>(cs->pages.size()) * c.page_size) return SLED_ERR_ARG;
  cudaSetDevice(c.device_index);
  std::vector<int32_t> slots(n_tokens);
  for (int i = 0; i < n_tokens; ++i) slots[i] = static_cast<int32_t>(e->kvm->slot_of(*cs, i));
  const size_t bytes = static_cast<size_t>(n_tokens) * c.n_kv_heads * c.head_dim * dtype_size(c.kv_dtype);
  int32_t* d_slots = nullptr;
  char* stage = nullptr;
  CU_TRY(cudaMalloc(reinterpret_cast<void**>(&d_slots), slots.size() * 4));
  if (cudaMalloc(reinterpret_cast<void**>(&stage), 2 * bytes) != cudaSuccess) { cudaFree(d_slots); return SLED_ERR_DEVICE; }
  cudaMemcpyAsync(d_slots, slots.data(), slots.size() * 4, cudaMemcpyHostToDevice, e->stream);
  launch_kv_gather(e->kpool + e->kv_layer_bytes * layer, d_slots, n_tokens, c.n_kv_heads, c.head_dim, c.page_size, stage, c.kv_dtype, e->stream);
  launch_kv_gather(e->vpool + e->kv_layer_bytes * layer, d_slots, n_tokens, c.n_kv_heads, c.head_dim, c.page_size, stage + bytes, c.kv_dtype, e->stream);
  cudaMemcpyAsync(K, stage, bytes, cudaMemcpyDeviceToHost, e->stream);
  cudaMemcpyAsync(V, stage + bytes, bytes, cudaMemcpyDeviceToHost, e->stream);
  cudaError_t err = cudaStreamSynchronize(e->stream);
  cudaFree(d_slots);
  cudaFree(stage);
  return err == cudaSuccess ? SLED_OK : SLED_ERR_DEVICE;
}

int sled_debug_copy_logits(sled_engine* e, float* dst, int32_t n_rows) {
  if (!e || !dst || n_rows <= 0 || n_rows > e->last_T) return SLED_ERR_ARG;
  cudaSetDevice(e->cfg.device_index);
  CU_TRY(cudaMemcpyAsync(dst, e->logits, static_cast<size_t>(n_rows) * e->cfg.vocab * 4, cudaMemcpyDefault, e->stream));
  CU_TRY(cudaStreamSynchronize(e->stream));
  return SLED_OK;
}

int sled_debug_truncate(sled_engine* e, uint64_t ctx_id, int64_t n_kv, int32_t pending) {
  if (!e || pending < 0 || pending >= e->cfg.vocab) return SLED_ERR_ARG;
  return e->kvm->truncate(ctx_id, n_kv, pending);
}

int sled_debug_truncate_batch(sled_engine* e, const uint64_t* ctx_ids, const int64_t* n_kv, const int32_t* pending,
                              int32_t n) {
  if (!e || n < 0 || (n > 0 && (!ctx_ids || !n_kv || !pending))) return SLED_ERR_ARG;
  for (int32_t i = 0; i < n; ++i) {
    const int rc = sled_debug_truncate(e, ctx_ids[i], n_kv[i], pending[i]);
    if (rc) return rc;
  }
  return SLED_OK;
}

int sled_debug_arm_wait_timeout(sled_engine* e, int32_t limit_us) {
  if (!e || !e->tc_error || limit_us <= 0 || limit_us > 100000) return SLED_ERR_ARG;
  e->probe_wait_cycles = static_cast<long long>(limit_us) * 2000;   // about 2 clock cycles per nanosecond
  return SLED_OK;
}

int sled_debug_set_commit(sled_engine* e, int32_t commit) {
  if (!e) return SLED_ERR_ARG;
  e->commit = commit != 0;
  return SLED_OK;
}

int sled_debug_set_timing(sled_engine* e, int32_t mode) {
  if (!e || mode < 0 || mode > 2) return SLED_ERR_ARG;
  cudaSetDevice(e->cfg.device_index);
  const size_t n = 16 + 20 * static_cast<size_t>(e->cfg.n_layers);   // launches (or kernel groups) of a step, with room to spare
  if (mode == 2 && e->ev_pool.empty()) {
    e->ev_pool.resize(n);
    e->ev_kind.assign(n, K_OTHER);
    for (auto& ev : e->ev_pool)
      if (cudaEventCreate(&ev) != cudaSuccess) return SLED_ERR_DEVICE;
  }
  if (mode == 1 && !e->d_stamps) {
    int rc = dmalloc(e, reinterpret_cast<void**>(&e->d_stamps), sizeof(unsigned long long) * 2 * n);
    if (rc) return rc;
    if (cudaMallocHost(reinterpret_cast<void**>(&e->h_stamps), sizeof(unsigned long long) * 2 * n) != cudaSuccess)
      return SLED_ERR_DEVICE;
    e->stamp_kind.assign(n, K_OTHER);
    e->stamp_cap = n;
  }
  e->timing = mode;
  return SLED_OK;
}

int sled_debug_shuffle_pages(sled_engine* e, uint64_t seed) {
  if (!e) return SLED_ERR_ARG;
  e->kvm->shuffle_free(seed);
  return SLED_OK;
}

int sled_debug_query_ctx(sled_engine* e, uint64_t ctx_id, int64_t* n_kv, int32_t* pending, int32_t* n_pages,
                         int32_t* pages_out, int32_t cap) {
  if (!e) return SLED_ERR_ARG;
  const CtxState* c = e->kvm->find(ctx_id);
  if (!c) return SLED_ERR_UNKNOWN_CTX;
  if (n_kv) *n_kv = c->n_kv;
  if (pending) *pending = c->pending;
  if (n_pages) *n_pages = static_cast<int32_t>(c->pages.size());
  if (pages_out)
    for (int32_t i = 0; i < cap && i < static_cast<int32_t>(c->pages.size()); ++i) pages_out[i] = c->pages[i];
  return SLED_OK;
}

}  // extern "C"

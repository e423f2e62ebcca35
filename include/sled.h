/*
 * sled.h -- C boundary of the batched verification step of SLED's edge server.
 *
 * The paper (Section 3.2) states the server's job: edge devices send the draft
 * tokens they generated, one shared target model verifies the drafts of many
 * devices together (Section 3.4), and each device gets back the position of its
 * first rejected token and the corrective token.  Acceptance follows Eq. 1 of
 * Section 3.1 (accept a draft x with probability min(1, p_target(x)/p_draft(x)),
 * on a rejection draw the replacement from the normalised positive part of
 * p_target - p_draft); when every draft is accepted one more token is drawn from
 * the target distribution that follows them.
 *
 * All entry points are plain C: fixed-width integers, raw pointers, an opaque
 * engine handle.  Unless a parameter says otherwise a pointer is a HOST pointer.
 * Every function returns SLED_OK (0) or a negative sled_status; a failed call
 * changes no context, page or counter.  An engine is used by one thread at a
 * time.  All device work is issued on the engine's stream, which does not wait for
 * any other stream: a DEVICE pointer passed in must refer to data that is already
 * complete (synchronise the stream that produced it first).
 */
#ifndef SLED_H_
#define SLED_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sled_engine sled_engine;
typedef struct sled_kvm sled_kvm;
typedef struct sled_planner sled_planner;

enum sled_status {
  SLED_OK = 0,
  SLED_ERR_ARG = -1,          /* null pointer, bad size, unsupported shape */
  SLED_ERR_UNKNOWN_CTX = -2,  /* ctx_id not open */
  SLED_ERR_DUP_CTX = -3,      /* ctx_id twice in one batch, or opened twice */
  SLED_ERR_K_RANGE = -4,      /* k < 0 or k > max_k */
  SLED_ERR_TOKEN_RANGE = -5,  /* token id outside [0, vocab) */
  SLED_ERR_NO_PAGES = -6,     /* KV pool exhausted */
  SLED_ERR_BATCH_TOO_LARGE = -7, /* n_reqs > max_batch or sum(k_i + 1) > max_step_tokens */
  SLED_ERR_NONFINITE = -8,    /* per-request status: a logit that had to be read was NaN or Inf */
  SLED_ERR_DEVICE = -9,       /* CUDA error, or a bounded device-side wait ran out */
  SLED_ERR_NO_DEVICE = -10,   /* no usable CUDA device: there is no CPU fallback */
  SLED_ERR_BASE_LEN = -11     /* base_len beyond the context's end, or before the start of its known token history */
};

/* returned by sled_poll while a request is still queued (not an error) */
#define SLED_PENDING 1

enum sled_dtype { SLED_F32 = 0, SLED_BF16 = 1 };

/* How the server forms batches (Section 3.4).  STATIC is the paper's scheme: requests wait until a fixed number
 * of them is there.  CONTINUOUS runs whatever has arrived, up to the capacity of a step. */
enum sled_batching { SLED_BATCH_STATIC = 0, SLED_BATCH_CONTINUOUS = 1 };

/* Shape of the Llama-style target model and the engine's capacities.
 * (The paper fixes only "Llama family", Section 4; shapes come from the workload.) */
typedef struct sled_config {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, ffn_dim, vocab;
  float rms_eps;          /* RMSNorm epsilon */
  float rope_theta;       /* rotary base; pairs (2i, 2i+1) rotate by pos * theta^(-2i/head_dim) */
  int32_t weight_dtype;   /* sled_dtype of every array in sled_weights; SLED_BF16 runs the linear
                             layers on the tensor cores with bf16 activations and fp32 accumulation,
                             SLED_F32 keeps everything in fp32 */
  int32_t kv_dtype;       /* sled_dtype of the cached keys and values */
  int32_t page_size;      /* tokens per KV page (16) */
  int32_t n_pages;        /* pages in the pool; one page holds page_size tokens of every layer */
  int32_t max_batch;      /* most requests per sled_verify_batch */
  int32_t max_k;          /* most draft tokens per request */
  int32_t max_step_tokens;/* most sum(k_i + 1) per step; also the prefill chunk */
  float temperature;      /* divides the target logits before the softmax (> 0) */
  int32_t greedy;         /* 1: accept iff the draft equals the argmax, emit the argmax */
  int32_t probs_on_device;/* 1: every sled_request.draft_probs will be a DEVICE pointer (no staging buffer is
                             allocated, host rows are then refused); 0: host or device, found out per request */
  int32_t device_index;   /* CUDA device ordinal */
  void* stream;           /* cudaStream_t to launch on; NULL: the engine creates one */
  int32_t draft_probs_dtype; /* sled_dtype of every sled_request.draft_probs row.  SLED_F32: exact.  SLED_BF16: rows
                             rounded to 16 bits by the device, half the bytes per request (Section 3.2 wants requests
                             small).  Eq. 1 is then applied with the rounded q: the output follows the target's
                             distribution up to the rounding of q (relative 2^-9 per entry), no longer exactly. */
  int32_t attention_impl; /* 0: the library's choice (the warp-level tensor-core kernel).  1: the tcgen05 kernel where it
                             applies (bf16 cache, 16-token pages, head_dim 128, requests of at most 48 query rows, i.e.
                             (k + 1) * n_q_heads / n_kv_heads <= 48); other steps fall back to 0.  Same results within
                             the attention tolerance; measured slower than 0 on the workloads here. */
  int32_t linear_weight_bits; /* 0 or 16: the linear layers' matrices are of weight_dtype.  8 (needs weight_dtype =
                             SLED_BF16): wq, wk, wv, wo, w_gate, w_up, w_down and lm_head are e4m3 bytes (1 sign, 4
                             exponent bits with bias 7, 3 mantissa bits, subnormals, no infinities; the patterns 0x7f and
                             0xff must not occur) and every output row has an fp32 scale: W[n][k] = scale[n] *
                             e4m3(byte[n][k]).  Half the weight bytes per step (the paper sweeps 16-, 8- and 4-bit
                             precision, Section 4).  The linear layers then run on fp8 tensor-core instructions, which
                             take both operands in 8 bits: every bf16 activation goes in as the sum of two e4m3 numbers
                             times a per-token scale - eight significant bits, as in bf16 - and the products are summed
                             in fp32; embedding, norms, attention and cache are as with 16-bit weights.  d_model, ffn_dim
                             and n_q_heads * head_dim must be multiples of 16.
                             4: the same with 4-bit weights - e2m1 codes (1 sign, 2 exponent bits with bias 1, 1 mantissa
                             bit: 0, 0.5, 1, 1.5, 2, 3, 4, 6 and their negatives), two to a byte, the even column in the
                             low half, rows of in/2 bytes: W[n][k] = scale[n] * e2m1(code[n][k]).  A quarter of the
                             weight bytes per step; only the weight operand of the fp8 instructions changes. */
} sled_config;

/* Target weights, row-major [out][in], all of type weight_dtype.  HOST or DEVICE
 * pointers (found out per pointer).  Copied during sled_init: the caller may free
 * them when it returns.  Per-layer members point to arrays of n_layers pointers. */
typedef struct sled_weights {
  const void* tok_emb;            /* [vocab][d_model] */
  const void* final_norm;         /* [d_model] */
  const void* lm_head;            /* [vocab][d_model] */
  const void* const* attn_norm;   /* [d_model] */
  const void* const* wq;          /* [n_q_heads*head_dim][d_model] */
  const void* const* wk;          /* [n_kv_heads*head_dim][d_model] */
  const void* const* wv;          /* [n_kv_heads*head_dim][d_model] */
  const void* const* wo;          /* [d_model][n_q_heads*head_dim] */
  const void* const* ffn_norm;    /* [d_model] */
  const void* const* w_gate;      /* [ffn_dim][d_model] */
  const void* const* w_up;        /* [ffn_dim][d_model] */
  const void* const* w_down;      /* [d_model][ffn_dim] */
  /* linear_weight_bits = 8 or 4 only (ignored otherwise): fp32 scales, one per output row of the matrix of the same name */
  const float* lm_head_scale;         /* [vocab] */
  const float* const* wq_scale;       /* [n_q_heads*head_dim] */
  const float* const* wk_scale;       /* [n_kv_heads*head_dim] */
  const float* const* wv_scale;       /* [n_kv_heads*head_dim] */
  const float* const* wo_scale;       /* [d_model] */
  const float* const* w_gate_scale;   /* [ffn_dim] */
  const float* const* w_up_scale;     /* [ffn_dim] */
  const float* const* w_down_scale;   /* [d_model] */
} sled_weights;

/* One device's verification request (Section 3.2: the draft tokens it sends;
 * Eq. 1 needs the draft model's distribution at each of them as well).  All
 * devices share the target's tokenizer (Section 3.4), so a row of draft_probs
 * has exactly `vocab` entries.  Borrowed for the duration of the call. */
typedef struct sled_request {
  uint64_t ctx_id;             /* context opened by sled_prefill */
  const int32_t* draft_tokens; /* [k], host */
  const void* draft_probs;     /* [k][vocab] of cfg.draft_probs_dtype (fp32 unless set otherwise), rows sum to 1; host
                                  (copied in during the forward pass) or device (read in place); may be NULL when
                                  k == 0 or in greedy mode */
  int32_t k;                   /* 0 <= k <= max_k; k = 0 is an ordinary decoding step */
  int64_t base_len;            /* 0: the drafts continue the context's current end.  m > 0: they continue its first m
                                  committed tokens - the length the device knew when it drafted.  Section 3.3: a device
                                  whose timer ran out sends its drafts again, extended; if the server had processed the
                                  first copy after all, it goes back to m before verifying, so the same request may be
                                  sent any number of times.  m may reach back as far as the context's tokens are known
                                  (everything for a context opened by sled_prefill) and not beyond its current end:
                                  SLED_ERR_BASE_LEN otherwise.  The cut is made once the whole call has passed
                                  validation and reservation; a device failure later leaves the context at m. */
} sled_request;

/* The feedback of Section 3.2: how many drafts were accepted (the first rejected
 * one is draft n_accepted + 1) and the corrective token, or the bonus token when
 * n_accepted == k. */
typedef struct sled_result {
  int32_t n_accepted;
  int32_t next_token;
  int32_t status;   /* SLED_OK or SLED_ERR_NONFINITE (then nothing of this request is committed) */
} sled_result;

typedef struct sled_stats {
  int64_t steps, requests, tokens_scored, drafts_accepted, tokens_committed;
  int32_t pages_total, pages_free, contexts_open;
  int64_t kernels_launched;    /* device kernels launched by this engine so far */
  int64_t kernels_last_step;   /* ... by the last sled_verify_batch */
  /* device time of the last step by kind of kernel, filled while sled_debug_set_timing is on; ms_idle: stretches of
   * the step in which no kernel ran (mode 1 only) */
  float ms_linear, ms_attention, ms_accept, ms_other, ms_step;
  int32_t linear_launches_last_step, attention_launches_last_step;
  float ms_idle;
} sled_stats;

/* ---- the three calls of the verification service ---------------------------------- */

/* Creates an engine around the one target model that all devices share (Section 3.2: the
 * server holds a single large model; Section 3.4: it verifies the drafts of many devices
 * together): checks cfg, allocates weights, KV pool and workspaces on
 * cfg->device_index, copies the weights.  Errors: SLED_ERR_ARG, SLED_ERR_NO_DEVICE,
 * SLED_ERR_DEVICE (allocation failed: nothing is left allocated). */
int sled_init(const sled_weights* w, const sled_config* cfg, sled_engine** out);

/* One batched verification step (Sections 3.1, 3.4).  For request i the target is
 * evaluated at the k_i + 1 tokens [pending_i, d_1..d_k] in one ragged pass over all
 * requests (no padding to a common length); draft j of context i is decided with the
 * Philox4x32-10 uniforms of (seed, ctx_id, absolute position of that token), so a
 * request's outcome does not depend on its batch slot or on the other requests.
 * Afterwards the KV entries of pending_i and of the accepted drafts are kept, those
 * of the rejected drafts are dropped, pages left empty return to the pool, and
 * next_token becomes the context's pending token.  results: caller-allocated [n_reqs].
 * All requests are validated and all pages reserved before anything changes. */
int sled_verify_batch(sled_engine* e, const sled_request* reqs, int32_t n_reqs, uint64_t seed,
                      sled_result* results);

/* Closes a context - a device's conversation has ended, or the device has left (Section 3.2:
 * each device is served on its own sequence) - and returns its pages to the pool.  The paper
 * leaves cache management to future work (Section 5); this call is what frees it here.
 * Errors: SLED_ERR_UNKNOWN_CTX. */
int sled_release(sled_engine* e, uint64_t ctx_id);

/* ---- what makes the three usable --------------------------------------------------- */

/* Opens a context from a device's prompt (Section 3.2: prompts are tokenised on the
 * device): caches the keys/values of tokens[0..n-2]; tokens[n-1] becomes the pending
 * token, fed first by the next verification.  n >= 1. */
int sled_prefill(sled_engine* e, uint64_t ctx_id, const int32_t* tokens, int32_t n);

int sled_set_sampling(sled_engine* e, float temperature, int32_t greedy);
int sled_get_stats(sled_engine* e, sled_stats* out);
/* cudaStream_t all work of this engine is issued on (for timing with events). */
void* sled_get_stream(sled_engine* e);
void sled_shutdown(sled_engine* e);
const char* sled_strerror(int status);

/* ---- the server loop around the step (Section 3.4, Fig. 2: queue -> batch planner -> target model) -------- */

/* Batching policy of sled_step; batch_size is the fixed size a STATIC batch waits for (<= max_batch; ignored by
 * CONTINUOUS, the default).  Only while nothing is queued. */
int sled_server_config(sled_engine* e, int32_t policy, int32_t batch_size);
/* Queues one device's request and returns a ticket for it.  The draft tokens are copied; req->draft_probs is
 * borrowed until the ticket's result has been polled.  Checked here: k, token ids, that the context is open. */
int sled_submit(sled_engine* e, const sled_request* req, uint64_t* ticket);
/* Lets the batch planner take the next batch out of the queue (arrival order; one request per context and step;
 * at most max_batch requests and max_step_tokens tokens - the paper pads a batch to a common length, here it is
 * ragged) and verifies it with sled_verify_batch.  STATIC: does nothing while fewer than batch_size requests wait,
 * unless flush != 0.  *n_verified (may be NULL): requests verified by this call.  A request whose context has been
 * released or cut back since it was queued gets its own error status and does not stop the others; if the step
 * itself fails, every request of the batch is answered with that code, which is also returned. */
int sled_step(sled_engine* e, uint64_t seed, int32_t flush, int32_t* n_verified);
/* SLED_OK and the result if the ticket's request has been verified (the ticket is then forgotten), SLED_PENDING
 * while it is queued, SLED_ERR_ARG for an unknown ticket. */
int sled_poll(sled_engine* e, uint64_t ticket, sled_result* out);
/* Requests waiting in the queue. */
int32_t sled_queued(sled_engine* e);

/* The queue and batch planner alone (host only, no device needed): what sled_submit / sled_step use. */
sled_planner* sled_planner_create(int32_t policy, int32_t batch_size, int32_t max_batch, int32_t max_step_tokens);
void sled_planner_destroy(sled_planner* p);
int sled_planner_push(sled_planner* p, uint64_t ticket, uint64_t ctx_id, int32_t k);
/* Next batch, whole or not at all: its tickets into tickets_out (cap entries); returns their number, 0 if no
 * batch is due, SLED_ERR_BATCH_TOO_LARGE (queue unchanged) if cap is too small. */
int32_t sled_planner_next_batch(sled_planner* p, int32_t flush, uint64_t* tickets_out, int32_t cap);
int32_t sled_planner_queued(sled_planner* p);

/* Host only: how a step's requests are cut into attention work items (request, KV head, chunk of keys) - the paper's
 * batched verification (Section 3.4) leaves the scheduling of the batch on the GPU open.  n_keys[i]: keys request i
 * attends to (cached prefix + its k_i + 1 new tokens), q_tokens[i] = k_i + 1, group: query heads per KV head,
 * resident_blocks: blocks of the attention kernel the GPU holds at once (two per SM), part_rows_cap: most rows of
 * partial results.  chunk_keys_out[i] (caller-allocated, n_reqs entries): keys per item of request i, a multiple of 64;
 * a request is cut into ceil(n_keys / chunk) equal parts.  Returns SLED_ERR_ARG on null pointers or non-positive sizes. */
int sled_debug_plan_attention(const int64_t* n_keys, const int32_t* q_tokens, int32_t n_reqs, int32_t n_kv_heads,
                              int32_t group, int32_t resident_blocks, int64_t part_rows_cap, int64_t* chunk_keys_out);

/* ---- stand-alone pieces of the step (device-resident operands) ---------------------- */

/* Acceptance only (Eq. 1 + residual / bonus draw) on logits already in device memory.
 *   logits   DEVICE [n_rows][vocab] fp32, request i owns rows cu_rows[i] .. cu_rows[i+1]-1
 *            (k_i + 1 rows: row j scores draft j+1, the last one the bonus token)
 *   cu_rows  HOST [n_reqs+1];  drafts HOST [n_rows - n_reqs] packed request after request
 *   q_rows   DEVICE [sum k_i][vocab] fp32 packed the same way (NULL if greedy)
 *   ctx_ids, pos0 HOST [n_reqs]: Philox counter words; pos0 = index of the pending token
 *   results  HOST [n_reqs]
 * stream: cudaStream_t or NULL for the default stream.  device_ms (may be NULL) receives the
 * kernel's duration measured with events on that stream.  Synchronises before returning. */
int sled_accept_rows(const float* logits, const int32_t* cu_rows, const int32_t* drafts, const float* q_rows,
                     const uint64_t* ctx_ids, const int64_t* pos0, int32_t n_reqs, int32_t vocab,
                     float temperature, int32_t greedy, uint64_t seed, sled_result* results, void* stream,
                     float* device_ms);

/* The same acceptance as sled_accept_rows for callers that must not allocate device memory
 * (the paper has no counterpart: this is a property of the library, not of the method).
 * A process whose GPU memory is wholly owned by another allocator, a latency path on which an
 * allocation would stall the device, or a caller between two points of a fixed schedule cannot
 * afford the cudaMalloc / cudaFree pair that sled_accept_rows performs for its small device-side
 * description of the batch.  Here that description lives in a fixed array inside the library
 * image: SLED_STATIC_MAX_REQS requests and SLED_STATIC_MAX_ROWS rows at most (just under 69 KB, held
 * by every GPU that loads the library until the process ends; the call also builds a host image
 * of that size on the caller's stack).  Larger batches are refused with
 * SLED_ERR_BATCH_TOO_LARGE.  The call allocates nothing on the device and nothing on the host
 * heap; it does not measure time.  Arguments and results are those of sled_accept_rows.
 * Every call must be made with the device that holds `logits` current (checked: SLED_ERR_ARG
 * otherwise).  The first call on a device looks up the array's device address; make that first
 * call before starting any stream capture, and from one thread.  All calls on a device share the one
 * array and every call rewrites it completely, so two calls must not overlap on the GPU: issue
 * them from one thread, one after the other (the call synchronises `stream` before returning). */
#define SLED_STATIC_MAX_REQS 1024
#define SLED_STATIC_MAX_ROWS 8192
int sled_accept_rows_static(const float* logits, const int32_t* cu_rows, const int32_t* drafts, const float* q_rows,
                            const uint64_t* ctx_ids, const int64_t* pos0, int32_t n_reqs, int32_t vocab,
                            float temperature, int32_t greedy, uint64_t seed, sled_result* results, void* stream);

/* Ragged verification attention only, over the engine's paged cache: request i's last
 * q_len[i] cached tokens are taken as the new ones; query j of request i attends to the
 * keys 0 .. n_kv_i - q_len_i + j of ctx_ids[i] in layer `layer`.
 *   q    DEVICE [sum q_len][n_q_heads][head_dim] in the activation type (bf16 with bf16 weights)
 *   out  DEVICE same shape and type.
 * device_ms (may be NULL) receives the duration of the attention kernels (events on the
 * engine's stream).  Synchronises before returning. */
int sled_attention_ragged(sled_engine* e, int32_t layer, const uint64_t* ctx_ids, const int32_t* q_len,
                          int32_t n_reqs, const void* q, void* out, float* device_ms);

/* ---- test and benchmark hooks ------------------------------------------------------- */

/* Opens a context with given cache content instead of a prefill.  K, V: HOST or DEVICE,
 * [n_layers][n_tokens][n_kv_heads][head_dim] of kv_dtype. */
int sled_debug_load_kv(sled_engine* e, uint64_t ctx_id, const void* K, const void* V, int32_t n_tokens,
                       int32_t pending);
/* Reads one layer's cache of a context back: K, V HOST [n_tokens][n_kv_heads][head_dim] of kv_dtype. */
int sled_debug_read_kv(sled_engine* e, uint64_t ctx_id, int32_t layer, void* K, void* V, int32_t n_tokens);
/* Copies the logits of the last step, rows [0, n_rows), to dst (HOST or DEVICE) [n_rows][vocab] fp32. */
int sled_debug_copy_logits(sled_engine* e, float* dst, int32_t n_rows);
/* Sets a context back to n_kv cached tokens (<= its current count) and a pending token. */
int sled_debug_truncate(sled_engine* e, uint64_t ctx_id, int64_t n_kv, int32_t pending);
/* The same for n contexts in one call (ctx_ids, n_kv, pending: HOST arrays [n]); stops at the first error. */
int sled_debug_truncate_batch(sled_engine* e, const uint64_t* ctx_ids, const int64_t* n_kv, const int32_t* pending,
                              int32_t n);
/* Self-test of the recovery from a device-side wait that runs out (engines with bf16 weights).  Every wait inside
 * the tensor-core and attention kernels is bounded: when one expires the kernel records a code, kernels that follow
 * return early, and sled_verify_batch returns SLED_ERR_DEVICE with every context, page and counter as before.  This
 * call arms that path without any fault: the next sled_verify_batch starts with a small kernel that waits limit_us
 * microseconds (<= 100000) on a barrier nobody signals, using the kernels' own bounded wait.  That step fails as
 * described; the one after it runs normally. */
int sled_debug_arm_wait_timeout(sled_engine* e, int32_t limit_us);
/* commit = 0: verification steps leave every context as it was (repeatable timing). */
int sled_debug_set_commit(sled_engine* e, int32_t commit);
/* Device time per kind of kernel into sled_stats.  mode 0: off.  mode 1: every launch stamps the GPU's global timer
 * when its first block begins and its last block ends; launches keep overlapping as they do untimed, and a launch
 * is charged the time by which it extends the step beyond all earlier launches (the parts add up to ms_step).
 * mode 2: CUDA events between kernel groups, which serialises neighbouring launches (each kernel's stand-alone
 * duration; the parts add up to more than an untimed step). */
int sled_debug_set_timing(sled_engine* e, int32_t mode);
/* Context state: cached tokens, pending token, owned pages (ids into pages_out, up to cap). */
int sled_debug_query_ctx(sled_engine* e, uint64_t ctx_id, int64_t* n_kv, int32_t* pending, int32_t* n_pages,
                         int32_t* pages_out, int32_t cap);

/* Permutes the free-page list (seeded), so contexts opened afterwards get physically scattered pages. */
int sled_debug_shuffle_pages(sled_engine* e, uint64_t seed);

/* ---- host-side KV page manager (no device needed) ----------------------------------- */
/* The bookkeeping the engine uses for commit / rollback, exported so it can be
 * exercised alone.  A context owns ceil(tokens / page_size) pages; pages are handed out
 * and returned whole; a batch reservation either fits entirely or changes nothing. */
sled_kvm* sled_kvm_create(int32_t n_pages, int32_t page_size);
void sled_kvm_destroy(sled_kvm* m);
int sled_kvm_open(sled_kvm* m, uint64_t ctx_id, int64_t n_kv, int32_t pending);
/* Reserves room for extra[i] more tokens behind the cached ones of each context. */
int sled_kvm_reserve_batch(sled_kvm* m, const uint64_t* ctx_ids, const int32_t* extra, int32_t n);
/* Keeps n_keep of the reserved tokens, returns pages that no longer hold any, sets pending. */
int sled_kvm_commit(sled_kvm* m, uint64_t ctx_id, int32_t n_keep, int32_t pending);
int sled_kvm_release(sled_kvm* m, uint64_t ctx_id);
int sled_kvm_query(sled_kvm* m, uint64_t ctx_id, int64_t* n_kv, int32_t* pending, int32_t* n_pages,
                   int32_t* pages_out, int32_t cap);
int32_t sled_kvm_free_pages(sled_kvm* m);
/* As sled_kvm_reserve_batch, with request i continuing the first base_len[i] committed tokens of its context
 * (0: its current end; see sled_request.base_len): the context is cut back first.  All or nothing. */
int sled_kvm_reserve_batch_at(sled_kvm* m, const uint64_t* ctx_ids, const int32_t* extra, const int64_t* base_len,
                              int32_t n);
/* As sled_kvm_commit, recording the kept tokens: kept[0 .. n_keep-2] are the tokens behind the old pending one
 * whose cache entries stay (the accepted drafts), then `pending`. */
int sled_kvm_commit_tokens(sled_kvm* m, uint64_t ctx_id, int32_t n_keep, int32_t pending, const int32_t* kept);
/* The known committed tokens of a context: they start at sequence index *hist_start, the last one is pending. */
int sled_kvm_history(sled_kvm* m, uint64_t ctx_id, int64_t* hist_start, int32_t* n_tokens, int32_t* tokens_out,
                     int32_t cap);
/* Ragged packing of one step: for request i with k[i] drafts, writes token rows
 * cu_q[i] .. cu_q[i+1]-1 (row 0 = pending token, then the drafts): ids, owning request,
 * absolute position and physical cache slot (page * page_size + offset).  Pages must have
 * been reserved.  Output arrays: cu_q [n+1], others [sum(k_i+1)]. */
int sled_kvm_pack(sled_kvm* m, const uint64_t* ctx_ids, const int32_t* k, const int32_t* const* drafts, int32_t n,
                  int32_t* cu_q, int32_t* ids, int32_t* tok_req, int32_t* tok_pos, int32_t* tok_slot);

#ifdef __cplusplus
}
#endif
#endif /* SLED_H_ */

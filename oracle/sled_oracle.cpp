// TEST INFRASTRUCTURE ONLY -- plain, slow CPU statement of SLED's batched
// verification step.  Nothing in the product path may include, link or call
// this file; it shares no code, header, table or constant generator with the
// CUDA library.  Every function cites the passage of the paper (or of the
// speculative-sampling method the paper adopts in Section 3.1) it follows.
//
// What is stated here:
//   * the Llama-style target forward, one token at a time (the k+1 positions
//     of a verification are k+1 single-token evaluations: scoring them in
//     one target pass, Section 3.1, is an execution strategy; the result is
//     defined by the autoregressive evaluation);
//   * the acceptance rule of Eq. 1 with residual resampling (Section 3.1) in
//     the fixed integer arithmetic that makes the decision independent of the
//     order in which a vocabulary row is reduced;
//   * Philox4x32-10 (Salmon et al., SC'11) from its published definition.
//
// Floating point: the forward runs in fp64 (weights are upcast exactly, K and
// V are rounded to the cache format when stored -- a property of the format),
// logits are rounded once to fp32; the acceptance arithmetic is the fixed
// fp32 / uint64 / fp64 sequence described at orc_fixed_exp / orc_accept.
//
// Parity pins live in tests/ (run with -m "not gpu"): Philox known answers and
// a second implementation, closed forms of the acceptance rule, the chi-square
// losslessness invariant, an independent library forward (both evaluation modes of
// orc_forward_token), and the bf16 rounding against a library conversion incl. ties.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------- formats --
inline double bf16_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return static_cast<double>(f);
}

// round-to-nearest-even to the bf16 grid; returned as a float holding that value
inline float round_to_bf16(double x) {
  float f = static_cast<float>(x);
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return f;  // inf / nan unchanged
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  u &= 0xffff0000u;
  std::memcpy(&f, &u, 4);
  return f;
}

struct Tensor {  // a weight array of either storage type, read as double
  const void* p;
  int dtype;  // 0 = fp32, 1 = bf16
  inline double at(int64_t i) const {
    return dtype == 0 ? static_cast<double>(static_cast<const float*>(p)[i])
                      : bf16_to_double(static_cast<const uint16_t*>(p)[i]);
  }
};

}  // namespace

extern "C" {

// The cache format's rounding, exposed so that tests can pin it against a library conversion.
float orc_round_bf16(double x) { return round_to_bf16(x); }

// ----------------------------------------------------------------- Philox --
// Philox4x32 with 10 rounds, as defined by Salmon, Moraes, Dror, Shaw,
// "Parallel random numbers: as easy as 1, 2, 3" (SC'11): multipliers
// 0xD2511F53 / 0xCD9E8D57, Weyl key increments 0x9E3779B9 / 0xBB67AE85.
void orc_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;
    uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
    uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = static_cast<uint32_t>(p1);
    uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = static_cast<uint32_t>(p0);
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The two uniforms of one decided position.  Key = the 64-bit seed, counter =
// (context id, absolute 0-based sequence index of the token being decided, 0):
// word 0 -> acceptance uniform (top 24 bits, u = U/2^24), word 1 -> sampling
// uniform (32 bits).  Keying by context and position rather than by batch slot
// makes a request's outcome independent of what else is in the batch.
void orc_uniforms(uint64_t seed, uint64_t ctx_id, int64_t abs_pos, uint32_t* u_acc24, uint32_t* u_smp32) {
  uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
  uint32_t ctr[4] = {static_cast<uint32_t>(ctx_id), static_cast<uint32_t>(ctx_id >> 32),
                     static_cast<uint32_t>(abs_pos), 0u};
  uint32_t w[4];
  orc_philox4x32_10(key, ctr, w);
  *u_acc24 = w[0] >> 8;
  *u_smp32 = w[1];
}

// ------------------------------------------------------ fixed-point softmax --
// E(x) = trunc(exp(x) * 2^40) for x <= 0 (x = scaled logit minus the row
// maximum), with exp evaluated by one fixed sequence of correctly rounded fp32
// operations so that every implementation gets the same integer:
//   x < -30            -> 0   (exp(x) * 2^40 < 1 there)
//   n  = rint(x*log2e) via the 1.5*2^23 shift (one fma, one subtract)
//   r  = fma(n, -ln2_hi, x); r = fma(n, -ln2_lo, r)
//   p  = degree-6 Taylor polynomial of exp(r), Horner form, fma at each step
//   E  = trunc(p * 2^(n+40)), an exact scaling of p's significand.
// Softmax numerators are these integers and the denominator is their exact
// uint64 sum, so p_v = E_v / Z carries no dependence on summation order.
uint64_t orc_fixed_exp(float x) {
  if (!(x >= -30.0f)) return 0;  // also catches NaN
  const float log2e = 0x1.715476p+0f, shift = 12582912.0f;
  const float ln2_hi = 0x1.62e4p-1f, ln2_lo = 0x1.7f7d1cp-20f;
  float t = fmaf(x, log2e, shift);
  float nf = t - shift;
  float r = fmaf(nf, -ln2_hi, x);
  r = fmaf(nf, -ln2_lo, r);
  float p = 0x1.6c16c2p-10f;           // 1/720
  p = fmaf(p, r, 0x1.111112p-7f);      // 1/120
  p = fmaf(p, r, 0x1.555556p-5f);      // 1/24
  p = fmaf(p, r, 0x1.555556p-3f);      // 1/6
  p = fmaf(p, r, 0.5f);
  p = fmaf(p, r, 1.0f);
  p = fmaf(p, r, 1.0f);
  int n = static_cast<int>(nf);
  uint32_t bits;
  std::memcpy(&bits, &p, 4);
  uint64_t mant = (bits & 0x7fffffu) | 0x800000u;
  int sh = (static_cast<int>(bits >> 23) - 127) + n + 40 - 23;
  if (sh >= 0) return mant << sh;
  if (sh > -24) return mant >> (-sh);
  return 0;
}

// Diagnostics of one request's decision: how close the deciding comparisons
// were, as relative changes of a probability (a logit change of d moves a
// probability by about a factor e^d).
struct orc_margin {
  double accept_rel;  // min over the accept tests taken of |lhs-rhs| / max(lhs, rhs)
  double sample_rel;  // distance of the sampling target to the nearer CDF boundary of the chosen token, / total weight
  double greedy_gap;  // smallest (top1 - top2) logit gap over the rows looked at (greedy mode)
  double draw_mass;   // total weight the token was drawn from, as a fraction of the row's Z (1 on a bonus row, the
                      // rejected mass sum max(p - q, 0) after a rejection): small values make the draw sensitive
};

enum { ORC_OK = 0, ORC_NONFINITE = 1 };

// Acceptance for ONE request (Section 3.1, Eq. 1, and the sentence after it).
//   logits : [k+1][V] fp32 target logits; row j-1 scores draft j, row k the bonus token
//   q      : [k][V] fp32 draft distributions (unused when greedy)
//   drafts : [k] draft token ids
//   pos0   : 0-based sequence index of the pending token (the first token fed),
//            so draft j is the token at index pos0 + j.
// Sampling mode, for j = 1..k:  accept draft j iff u_j < p_j(d_j) / q_j(d_j)
// (the min(1, .) of Eq. 1 changes nothing since u_j < 1).  At the first
// rejection r the corrective token is drawn from norm(max(p_r - q_r, 0)): the
// paper gives the residual as the plain difference of the two distributions;
// it is made a distribution the way the method it cites does (clip at zero,
// normalise).  With no rejection a bonus token is drawn from
// p_{k+1}.  All in the fixed arithmetic:
//   s_v = z_v * (1/tau) (one fp32 multiply), m = max s_v, E_v = E(s_v - m), Z = sum E_v
//   accept  <=>  (double(U) * double(q_d)) * double(Z)  <  double(E_d) * 2^24
//   R_v = max(E_v - trunc(double(q_v) * double(Z)), 0),  W = sum R_v   (W = 0 -> R = E)
//   tgt = (U' * W) >> 32,  next = min{ v : sum_{w<=v} R_w > tgt }
// Greedy mode: accept iff d_j equals the lowest-index argmax of row j-1.
// A non-finite logit in a row that is looked at gives ORC_NONFINITE with
// n_accepted = 0 and next = -1.
int orc_accept(const float* logits, const float* q, const int32_t* drafts, int32_t k, int32_t V,
               float tau, int32_t greedy, uint64_t seed, uint64_t ctx_id, int64_t pos0,
               int32_t* n_accepted, int32_t* next_token, orc_margin* mg) {
  orc_margin local = {INFINITY, INFINITY, INFINITY, 1.0};
  const float inv_tau = 1.0f / tau;
  std::vector<uint64_t> E(static_cast<size_t>(V));
  *n_accepted = 0;
  *next_token = -1;
  for (int32_t j = 0; j <= k; ++j) {  // row j decides draft j+1, or is the bonus row when j == k
    const float* z = logits + static_cast<int64_t>(j) * V;
    for (int32_t v = 0; v < V; ++v)
      if (!std::isfinite(z[v])) { if (mg) *mg = local; *n_accepted = 0; *next_token = -1; return ORC_NONFINITE; }
    if (greedy) {
      int32_t best = 0;
      for (int32_t v = 1; v < V; ++v) if (z[v] > z[best]) best = v;
      float second = -INFINITY;
      for (int32_t v = 0; v < V; ++v) if (v != best && z[v] > second) second = z[v];
      double gap = static_cast<double>(z[best]) - static_cast<double>(second);
      if (gap < local.greedy_gap) local.greedy_gap = gap;
      if (j < k && drafts[j] == best) continue;  // accepted, look at the next row
      *n_accepted = j;
      *next_token = best;
      if (mg) *mg = local;
      return ORC_OK;
    }
    // fixed-point softmax numerators of this row
    float m = -INFINITY;
    for (int32_t v = 0; v < V; ++v) { float s = z[v] * inv_tau; if (s > m) m = s; }
    uint64_t Z = 0;
    for (int32_t v = 0; v < V; ++v) { float s = z[v] * inv_tau; E[v] = orc_fixed_exp(s - m); Z += E[v]; }
    uint32_t u_acc, u_smp;
    orc_uniforms(seed, ctx_id, pos0 + j + 1, &u_acc, &u_smp);
    const float* qrow = nullptr;
    if (j < k) {
      qrow = q + static_cast<int64_t>(j) * V;
      int32_t d = drafts[j];
      double lhs = (static_cast<double>(u_acc) * static_cast<double>(qrow[d])) * static_cast<double>(Z);
      double rhs = static_cast<double>(E[d]) * 16777216.0;
      double big = lhs > rhs ? lhs : rhs;
      double rel = big > 0 ? std::fabs(lhs - rhs) / big : 0.0;
      if (rel < local.accept_rel) local.accept_rel = rel;
      if (lhs < rhs) continue;  // accepted
    }
    // decision row: residual (after a rejection) or plain p (bonus)
    uint64_t W = 0;
    std::vector<uint64_t> R(static_cast<size_t>(V));
    if (qrow) {
      for (int32_t v = 0; v < V; ++v) {
        uint64_t Q = static_cast<uint64_t>(static_cast<double>(qrow[v]) * static_cast<double>(Z));
        R[v] = E[v] > Q ? E[v] - Q : 0;
        W += R[v];
      }
    }
    if (W == 0) { for (int32_t v = 0; v < V; ++v) R[v] = E[v]; W = Z; }
    uint64_t tgt = static_cast<uint64_t>((static_cast<unsigned __int128>(u_smp) * W) >> 32);
    uint64_t run = 0;
    int32_t pick = V - 1;
    for (int32_t v = 0; v < V; ++v) {
      uint64_t before = run;
      run += R[v];
      if (run > tgt) {
        pick = v;
        double lo = static_cast<double>(tgt - before), hi = static_cast<double>(run - tgt);
        local.sample_rel = (lo < hi ? lo : hi) / static_cast<double>(W);
        local.draw_mass = static_cast<double>(W) / static_cast<double>(Z);
        break;
      }
    }
    *n_accepted = j;
    *next_token = pick;
    if (mg) *mg = local;
    return ORC_OK;
  }
  return ORC_OK;  // not reached: row k always decides
}

// Fixed-point softmax of one row, exposed so tests can pin it (sum and values).
void orc_fixed_softmax(const float* z, int32_t V, float tau, uint64_t* E_out, uint64_t* Z_out) {
  const float inv_tau = 1.0f / tau;
  float m = -INFINITY;
  for (int32_t v = 0; v < V; ++v) { float s = z[v] * inv_tau; if (s > m) m = s; }
  uint64_t Z = 0;
  for (int32_t v = 0; v < V; ++v) { float s = z[v] * inv_tau; E_out[v] = orc_fixed_exp(s - m); Z += E_out[v]; }
  *Z_out = Z;
}

// ------------------------------------------------------------ target model --
// Llama-style decoder: RMSNorm, rotary embedding on adjacent pairs, grouped-
// query attention, SwiGLU; no biases; separate embedding and LM head.  The
// paper only says the target is of the Llama family (Section 4); the shapes
// are those of the workloads.
struct orc_config {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, ffn_dim, vocab;
  float rms_eps, rope_theta;
  int32_t weight_dtype;  // 0 = fp32, 1 = bf16 (storage of every weight array)
  int32_t kv_dtype;      // 0 = fp32, 1 = bf16 (format K and V are rounded to when cached)
};

struct orc_weights {  // row-major [out][in]; per-layer arrays have n_layers entries
  const void* tok_emb;     // [vocab][d]
  const void* final_norm;  // [d]
  const void* lm_head;     // [vocab][d]
  const void* const* attn_norm;  // [d]
  const void* const* wq;         // [Hq*h][d]
  const void* const* wk;         // [Hkv*h][d]
  const void* const* wv;         // [Hkv*h][d]
  const void* const* wo;         // [d][Hq*h]
  const void* const* ffn_norm;   // [d]
  const void* const* w_gate;     // [F][d]
  const void* const* w_up;       // [F][d]
  const void* const* w_down;     // [d][F]
};

// y = W x, W row-major [n_out][n_in]; each output is one left-to-right fp64 sum
static void matvec(const Tensor& W, int64_t n_out, int64_t n_in, const double* x, double* y) {
#pragma omp parallel for schedule(static)
  for (int64_t o = 0; o < n_out; ++o) {
    double acc = 0.0;
    if (W.dtype == 0) {
      const float* row = static_cast<const float*>(W.p) + o * n_in;
      for (int64_t i = 0; i < n_in; ++i) acc += static_cast<double>(row[i]) * x[i];
    } else {
      const uint16_t* row = static_cast<const uint16_t*>(W.p) + o * n_in;
      for (int64_t i = 0; i < n_in; ++i) acc += bf16_to_double(row[i]) * x[i];
    }
    y[o] = acc;
  }
}

static void rmsnorm(const double* x, const Tensor& g, int64_t d, double eps, double* y) {
  double ss = 0.0;
  for (int64_t i = 0; i < d; ++i) ss += x[i] * x[i];
  double scale = 1.0 / std::sqrt(ss / static_cast<double>(d) + eps);
  for (int64_t i = 0; i < d; ++i) y[i] = x[i] * scale * g.at(i);
}

// rotate pairs (2i, 2i+1) of every head by pos * theta^(-2i/h)
static void rope(double* v, int n_heads, int h, int64_t pos, double theta) {
  for (int hd = 0; hd < n_heads; ++hd)
    for (int i = 0; i < h / 2; ++i) {
      double ang = static_cast<double>(pos) * std::pow(theta, -2.0 * i / static_cast<double>(h));
      double c = std::cos(ang), s = std::sin(ang);
      double a = v[hd * h + 2 * i], b = v[hd * h + 2 * i + 1];
      v[hd * h + 2 * i] = a * c - b * s;
      v[hd * h + 2 * i + 1] = a * s + b * c;
    }
}

static void round_vec(double* v, int64_t n) {
  for (int64_t i = 0; i < n; ++i) v[i] = static_cast<double>(round_to_bf16(v[i]));
}

// One token through the whole model.  kcache / vcache: [n_layers][cap][Hkv][h]
// floats holding values already rounded to the cache format, rows 0..pos-1
// filled; row pos is written here.  logits_out: [vocab] fp32.
// Returns 0, or -1 if pos >= cap.
//
// round_acts = 0 is the reference evaluation.  round_acts = 1 is a second, separately reported mode for
// the 16-bit configurations: every vector that a 16-bit implementation has to hand to a matrix product
// in 16 bits (the two normalised inputs of a layer, the rotated query, the attention output, the SwiGLU
// output, the final normalised vector) is rounded to bf16 at that point and nowhere else.  Comparing
// against it separates rounding of the activations, which grows with depth, from everything else.
int orc_forward_token(const orc_config* cfg, const orc_weights* w, int32_t token, int64_t pos,
                      float* kcache, float* vcache, int64_t cap, float* logits_out, int32_t round_acts) {
  const int L = cfg->n_layers, d = cfg->d_model, Hq = cfg->n_q_heads, Hkv = cfg->n_kv_heads;
  const int h = cfg->head_dim, F = cfg->ffn_dim, V = cfg->vocab, wd = cfg->weight_dtype;
  if (pos >= cap || pos < 0) return -1;
  const int group = Hq / Hkv;
  std::vector<double> x(d), a(d), qv(static_cast<size_t>(Hq) * h), kv(static_cast<size_t>(Hkv) * h),
      vv(static_cast<size_t>(Hkv) * h), o(static_cast<size_t>(Hq) * h), tmp(d), g(F), u(F);
  Tensor emb{w->tok_emb, wd};
  for (int i = 0; i < d; ++i) x[i] = emb.at(static_cast<int64_t>(token) * d + i);
  const int64_t layer_stride = cap * Hkv * h;
  for (int l = 0; l < L; ++l) {
    rmsnorm(x.data(), Tensor{w->attn_norm[l], wd}, d, cfg->rms_eps, a.data());
    if (round_acts) round_vec(a.data(), d);
    matvec(Tensor{w->wq[l], wd}, static_cast<int64_t>(Hq) * h, d, a.data(), qv.data());
    matvec(Tensor{w->wk[l], wd}, static_cast<int64_t>(Hkv) * h, d, a.data(), kv.data());
    matvec(Tensor{w->wv[l], wd}, static_cast<int64_t>(Hkv) * h, d, a.data(), vv.data());
    rope(qv.data(), Hq, h, pos, cfg->rope_theta);
    rope(kv.data(), Hkv, h, pos, cfg->rope_theta);
    if (round_acts) round_vec(qv.data(), static_cast<int64_t>(Hq) * h);
    float* kc = kcache + l * layer_stride;
    float* vc = vcache + l * layer_stride;
    for (int i = 0; i < Hkv * h; ++i) {
      kc[pos * Hkv * h + i] = cfg->kv_dtype == 1 ? round_to_bf16(kv[i]) : static_cast<float>(kv[i]);
      vc[pos * Hkv * h + i] = cfg->kv_dtype == 1 ? round_to_bf16(vv[i]) : static_cast<float>(vv[i]);
    }
    const double scale = 1.0 / std::sqrt(static_cast<double>(h));
#pragma omp parallel for schedule(static)
    for (int hd = 0; hd < Hq; ++hd) {
      const int kvh = hd / group;
      std::vector<double> sc(static_cast<size_t>(pos) + 1);
      double mx = -INFINITY;
      for (int64_t t = 0; t <= pos; ++t) {
        double dot = 0.0;
        const float* kr = kc + (t * Hkv + kvh) * h;
        for (int i = 0; i < h; ++i) dot += qv[static_cast<size_t>(hd) * h + i] * static_cast<double>(kr[i]);
        sc[t] = dot * scale;
        if (sc[t] > mx) mx = sc[t];
      }
      double den = 0.0;
      for (int64_t t = 0; t <= pos; ++t) { sc[t] = std::exp(sc[t] - mx); den += sc[t]; }
      for (int i = 0; i < h; ++i) {
        double acc = 0.0;
        for (int64_t t = 0; t <= pos; ++t) acc += sc[t] * static_cast<double>(vc[(t * Hkv + kvh) * h + i]);
        o[static_cast<size_t>(hd) * h + i] = acc / den;
      }
    }
    if (round_acts) round_vec(o.data(), static_cast<int64_t>(Hq) * h);
    matvec(Tensor{w->wo[l], wd}, d, static_cast<int64_t>(Hq) * h, o.data(), tmp.data());
    for (int i = 0; i < d; ++i) x[i] += tmp[i];
    rmsnorm(x.data(), Tensor{w->ffn_norm[l], wd}, d, cfg->rms_eps, a.data());
    if (round_acts) round_vec(a.data(), d);
    matvec(Tensor{w->w_gate[l], wd}, F, d, a.data(), g.data());
    matvec(Tensor{w->w_up[l], wd}, F, d, a.data(), u.data());
    for (int i = 0; i < F; ++i) g[i] = (g[i] / (1.0 + std::exp(-g[i]))) * u[i];
    if (round_acts) round_vec(g.data(), F);
    matvec(Tensor{w->w_down[l], wd}, d, F, g.data(), tmp.data());
    for (int i = 0; i < d; ++i) x[i] += tmp[i];
  }
  rmsnorm(x.data(), Tensor{w->final_norm, wd}, d, cfg->rms_eps, a.data());
  if (round_acts) round_vec(a.data(), d);
  std::vector<double> lg(static_cast<size_t>(V));
  matvec(Tensor{w->lm_head, wd}, V, d, a.data(), lg.data());
  for (int v = 0; v < V; ++v) logits_out[v] = static_cast<float>(lg[v]);
  return 0;
}

// Attention of one query head over a given cache prefix, exposed for the
// attention-only workload: q [h] (already rotated), keys/values [n][h] floats.
void orc_attend_one(const float* q, const float* keys, const float* values, int64_t n, int32_t h, double* out) {
  const double scale = 1.0 / std::sqrt(static_cast<double>(h));
  std::vector<double> sc(static_cast<size_t>(n));
  double mx = -INFINITY;
  for (int64_t t = 0; t < n; ++t) {
    double dot = 0.0;
    for (int i = 0; i < h; ++i) dot += static_cast<double>(q[i]) * static_cast<double>(keys[t * h + i]);
    sc[t] = dot * scale;
    if (sc[t] > mx) mx = sc[t];
  }
  double den = 0.0;
  for (int64_t t = 0; t < n; ++t) { sc[t] = std::exp(sc[t] - mx); den += sc[t]; }
  for (int i = 0; i < h; ++i) {
    double acc = 0.0;
    for (int64_t t = 0; t < n; ++t) acc += sc[t] * static_cast<double>(values[t * h + i]);
    out[i] = acc / den;
  }
}

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void orc_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

}  // extern "C"

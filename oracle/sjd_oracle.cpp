// CPU oracle for the SJD / SJD++ verify-and-redraft step.  TEST INFRASTRUCTURE ONLY: see the
// header for the rules that keep it apart from the CUDA library.  Plain loops, library sort and
// exp, double precision for the softmax; nothing here is blocked, fused or tuned.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -shared -fPIC sjd_oracle.cpp -o libsjd_oracle.so -lpthread
#include "sjd_oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3").
// One round: two 32x32->64 multiplies of counter words 0 and 2 by fixed odd constants; the high
// halves are xored with the other counter words and the round key, the low halves pass through
// with the words permuted.  The key is advanced by the golden-ratio / sqrt(3) Weyl constants
// between rounds.  Ten rounds.
// ---------------------------------------------------------------------------------------------
void philox_round(uint32_t c[4], const uint32_t k[2]) {
  const uint64_t prod0 = (uint64_t)0xD2511F53u * c[0];
  const uint64_t prod1 = (uint64_t)0xCD9E8D57u * c[2];
  const uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
  const uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
  const uint32_t n0 = hi1 ^ c[1] ^ k[0];
  const uint32_t n1 = lo1;
  const uint32_t n2 = hi0 ^ c[3] ^ k[1];
  const uint32_t n3 = lo0;
  c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void philox(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
  uint32_t k[2] = {key[0], key[1]};
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
    philox_round(c, k);
  }
  for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// The random numbers of one decision: counter = (position, batch, iteration, purpose),
// key = (seed low word, seed high word).
void draw(uint64_t seed, int32_t pos, int32_t b, int32_t iter, int32_t purpose, uint32_t out[4]) {
  const uint32_t ctr[4] = {(uint32_t)pos, (uint32_t)b, (uint32_t)iter, (uint32_t)purpose};
  const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
  philox(ctr, key, out);
}

float uniform24(uint32_t x) { return (float)(x >> 8) * (1.0f / 16777216.0f); }

// IEEE 754 binary16: 1 sign bit, 5 exponent bits (bias 15), 10 fraction bits.  Every value is exactly
// representable in fp32; written out case by case.
float half_to_float(uint16_t h) {
  const int sign = (h >> 15) & 1, e = (h >> 10) & 31, f = h & 1023;
  double v;
  if (e == 0) v = std::ldexp((double)f, -24);                  // zero and subnormals: f * 2^-10 * 2^-14
  else if (e == 31) v = f == 0 ? (double)INFINITY : (double)NAN;
  else v = std::ldexp(1.0 + (double)f / 1024.0, e - 15);
  return (float)(sign ? -v : v);
}

// bf16 -> fp32 is exact: the 16 bits are the upper half of the fp32 pattern.
float load_logit(const void* base, int32_t dtype, int64_t idx) {
  if (dtype == ORC_F16) return half_to_float(((const uint16_t*)base)[idx]);
  if (dtype == ORC_BF16) {
    const uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16;
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
  }
  return ((const float*)base)[idx];
}

// Section 3.1 sampling head for one row.  Guidance on logits (merged = u + s (c - u)), then the
// temperature, then top-K on the scaled logits, then softmax over the survivors only.
// fp32 with one rounding per operation for the merge (it decides the top-K SET, an integer
// decision), double for the exponentials and their sum.
int32_t row_probs(const void* cond, const void* uncond, int32_t dtype, int64_t off, int32_t V, float s,
                  float inv_T, int32_t top_k, int32_t* ids, float* vals, int32_t* degenerate) {
  if (V <= 0 || top_k < 1) return -1;
  const int32_t kcap = std::min(top_k, V);
  std::vector<float> y((size_t)V);
  for (int32_t v = 0; v < V; ++v) {
    const float c = load_logit(cond, dtype, off + v);
    float g = c;
    if (uncond != nullptr) {
      const float u = load_logit(uncond, dtype, off + v);
      const float d = c - u;      // rounded once
      g = std::fmaf(s, d, u);     // rounded once
    }
    float yv = g * inv_T;         // rounded once
    if (std::isnan(yv)) yv = -std::numeric_limits<float>::infinity();  // NaN ranks as masked
    y[(size_t)v] = yv;
  }
  // top-K: order by (y descending, id ascending) and keep the first kcap.
  std::vector<int32_t> order((size_t)V);
  for (int32_t v = 0; v < V; ++v) order[(size_t)v] = v;
  std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
    if (y[(size_t)a] != y[(size_t)b]) return y[(size_t)a] > y[(size_t)b];
    return a < b;
  });
  std::vector<int32_t> keep(order.begin(), order.begin() + kcap);
  std::sort(keep.begin(), keep.end());
  // softmax over the survivors
  double m = -std::numeric_limits<double>::infinity();
  for (int32_t k = 0; k < kcap; ++k) m = std::max(m, (double)y[(size_t)keep[(size_t)k]]);
  std::vector<double> e((size_t)kcap);
  double Z = 0.0;
  for (int32_t k = 0; k < kcap; ++k) {
    const double yk = (double)y[(size_t)keep[(size_t)k]];
    e[(size_t)k] = std::isinf(yk) && yk < 0 ? 0.0 : std::exp(yk - m);
    Z += e[(size_t)k];
  }
  const bool degen = !(Z > 0.0) || std::isinf(m);
  if (degenerate) *degenerate = degen ? 1 : 0;
  for (int32_t k = 0; k < kcap; ++k) {
    ids[k] = keep[(size_t)k];
    vals[k] = degen ? 0.0f : (float)(e[(size_t)k] / Z);
  }
  return kcap;
}

// p(token) on a sparse row: binary search in the ascending ids.
float lookup(const int32_t* ids, const float* vals, int32_t cnt, int32_t V, int32_t token) {
  if (cnt == ORC_Q_UNIFORM) return (token >= 0 && token < V) ? 1.0f / (float)V : 0.0f;
  const int32_t* end = ids + cnt;
  const int32_t* it = std::lower_bound(ids, end, token);
  if (it != end && *it == token) return vals[it - ids];
  return 0.0f;
}

// Eq. acc-sjdpp: accept iff r < min(1, p/q).  p == 0 can never be accepted (ratio 0, r >= 0);
// a non-positive q with p > 0 is an infinite ratio.
int32_t accept(float p_tok, float q_tok, float u, float* ratio_out) {
  float ratio;
  if (p_tok == 0.0f) ratio = 0.0f;
  else if (!(q_tok > 0.0f)) ratio = std::numeric_limits<float>::infinity();
  else ratio = p_tok / q_tok;  // fp32 division
  if (ratio_out) *ratio_out = ratio;
  const float bound = ratio < 1.0f ? ratio : 1.0f;
  return u < bound ? 1 : 0;
}

// Fixed-point inverse CDF, independent of summation order because every partial sum is exact.
int32_t icdf(const float* w, int32_t n, uint64_t R, float* margin_out) {
  const float scale = 1099511627776.0f;  // 2^40
  std::vector<uint64_t> Wk((size_t)std::max(n, 0));
  uint64_t T = 0;
  for (int32_t k = 0; k < n; ++k) {
    const float wk = w[k] > 0.0f ? w[k] : 0.0f;
    Wk[(size_t)k] = (uint64_t)(wk * scale);  // exact product, truncation toward zero
    T += Wk[(size_t)k];
  }
  if (margin_out) *margin_out = 0.0f;
  if (T == 0) return -1;
  const uint64_t t = (uint64_t)(((unsigned __int128)R * (unsigned __int128)T) >> 64);
  uint64_t below = 0;
  for (int32_t k = 0; k < n; ++k) {
    const uint64_t upto = below + Wk[(size_t)k];
    if (upto > t) {
      if (margin_out) {
        const uint64_t dlo = t - below, dhi = upto - t;
        *margin_out = (float)((double)std::min(dlo, dhi) / 1099511627776.0);
      }
      return k;
    }
    below = upto;
  }
  return n - 1;  // unreachable: t < T
}

void residual_weights(const int32_t* p_ids, const float* p_vals, int32_t p_cnt, const int32_t* q_ids,
                      const float* q_vals, int32_t q_cnt, int32_t V, float* w) {
  for (int32_t k = 0; k < p_cnt; ++k) {
    const float q = lookup(q_ids, q_vals, q_cnt, V, p_ids[k]);
    const float d = p_vals[k] - q;  // fp32 subtraction, Eq. rej-sjd numerator
    w[k] = d > 0.0f ? d : 0.0f;
  }
}

uint64_t r64(const uint32_t x[4]) { return (uint64_t)x[0] | ((uint64_t)x[1] << 32); }

struct StepCtx {
  const void* cond; const void* uncond; const int32_t* drafts; const orc_probs* q; const orc_params* P;
  uint64_t seed; int32_t* out_accept_len; int32_t* out_tokens; orc_probs* out; int32_t* out_flags;
  int32_t* status; orc_diag* diag; int32_t kcap;
};

int32_t seq_len(const StepCtx& c, int32_t b) {
  int32_t L = c.P->win_len ? c.P->win_len[b] : c.P->W;
  return std::max(0, std::min(L, c.P->W));
}

// Phase 1: the distribution of every valid row (Step 2 output turned into p_i).
void rows_phase(const StepCtx& c, int64_t row_begin, int64_t row_end, std::vector<int32_t>* degen) {
  const orc_params& P = *c.P;
  for (int64_t r = row_begin; r < row_end; ++r) {
    const int32_t b = (int32_t)(r / P.W), i = (int32_t)(r % P.W);
    int32_t* ids = c.out->ids + (size_t)r * c.kcap;
    float* vals = c.out->vals + (size_t)r * c.kcap;
    if (i >= seq_len(c, b)) {
      c.out->cnt[r] = 0;
      continue;
    }
    const int64_t off = (int64_t)b * P.stride_b + (int64_t)i * P.stride_w;
    int32_t dg = 0;
    c.out->cnt[r] = row_probs(c.cond, c.uncond, P.logits_dtype, off, P.V, P.cfg_scale, P.inv_temperature,
                              P.top_k, ids, vals, &dg);
    (*degen)[(size_t)r] = dg;
  }
}

// Phase 2: Steps 3 and 4 for one sequence.
void verify_phase(const StepCtx& c, int32_t b, const std::vector<int32_t>& degen) {
  const orc_params& P = *c.P;
  const int32_t W = P.W, V = P.V, L = seq_len(c, b);
  const int32_t pos0 = P.pos_base ? P.pos_base[b] : 0;
  const int32_t iter = P.iteration ? P.iteration[b] : P.iteration0;
  const int32_t gb = P.seq_base + b;  // sequence word of the counter
  const bool draft_all = (P.flags & ORC_FLAG_DRAFT_ALL) != 0;
  const bool reuse_on = (P.flags & ORC_FLAG_REUSE) != 0;
  int32_t st = 0;
  const size_t base = (size_t)b * W;

  std::vector<int32_t> ok((size_t)W, 0), reuse((size_t)W, 0), redraft_tok((size_t)W, -1);
  std::vector<float> ptok((size_t)W, 0.f), ratio((size_t)W, 0.f), redraft_p((size_t)W, 0.f);

  for (int32_t i = 0; i < L; ++i) {
    const size_t r = base + i;
    const int32_t* ids = c.out->ids + r * c.kcap;
    const float* vals = c.out->vals + r * c.kcap;
    const int32_t cnt = c.out->cnt[r];
    if (degen[r]) st |= ORC_STATUS_DEGENERATE_ROW;
    uint32_t x[4];
    if (!draft_all) {
      // Step 3: r < min(1, p_j(x_i) / p_{j-1}(x_i))
      const int32_t tok = c.drafts[r];
      const float qt = c.q->tok_prob[r];
      ptok[(size_t)i] = lookup(ids, vals, cnt, V, tok);
      draw(c.seed, pos0 + i, gb, iter, ORC_PURPOSE_ACCEPT, x);
      const float u = uniform24(x[0]);
      if (!(qt > 0.0f)) st |= ORC_STATUS_QTOK_NONPOSITIVE;
      ok[(size_t)i] = accept(ptok[(size_t)i], qt, u, &ratio[(size_t)i]);
      // confidence C_i of Eq. (C): the same ratio; reuse iff C_i > tau.  A draft with p_j(x_i) = 0
      // lies outside the current top-K support and is never kept, whatever tau is.
      reuse[(size_t)i] = (reuse_on && ptok[(size_t)i] > 0.0f && ratio[(size_t)i] > P.reuse_tau) ? 1 : 0;
      if (c.diag) {
        if (c.diag->u) c.diag->u[r] = u;
        if (c.diag->ratio) c.diag->ratio[r] = ratio[(size_t)i];
        if (c.diag->accept_margin) c.diag->accept_margin[r] = std::fabs(u - ratio[(size_t)i]);
        if (c.diag->reuse_margin) c.diag->reuse_margin[r] = std::fabs(ratio[(size_t)i] - P.reuse_tau);
        if (c.diag->pot_ok) c.diag->pot_ok[r] = ok[(size_t)i];
        if (c.diag->pot_reuse) c.diag->pot_reuse[r] = reuse[(size_t)i];
      }
    }
    // what the row would get if resampled from its current distribution (Eq. reuse, second case;
    // Eq. refine-sjd); evaluated for every row because the draw depends only on the row's counter
    draw(c.seed, pos0 + i, gb, iter, draft_all ? ORC_PURPOSE_INIT : ORC_PURPOSE_REDRAFT, x);
    float mg = 0.f;
    int32_t k = icdf(vals, cnt, r64(x), &mg);
    if (k < 0) k = 0;
    redraft_tok[(size_t)i] = ids[k];
    redraft_p[(size_t)i] = vals[k];
    if (c.diag) {
      if (c.diag->pot_redraft) c.diag->pot_redraft[r] = ids[k];
      if (c.diag->redraft_margin) c.diag->redraft_margin[r] = mg;
    }
  }

  // residual sample of Eq. rej-sjd for row i
  auto residual_at = [&](int32_t i, int32_t* tok, float* prob, float* margin, bool* empty) {
    const size_t r = base + i;
    const int32_t* ids = c.out->ids + r * c.kcap;
    const float* vals = c.out->vals + r * c.kcap;
    const int32_t cnt = c.out->cnt[r];
    std::vector<float> w((size_t)cnt);
    residual_weights(ids, vals, cnt, c.q->ids + r * c.kcap, c.q->vals + r * c.kcap, c.q->cnt[r], V, w.data());
    uint32_t x[4];
    draw(c.seed, pos0 + i, gb, iter, ORC_PURPOSE_RESIDUAL, x);
    int32_t k = icdf(w.data(), cnt, r64(x), margin);
    *empty = false;
    if (k < 0) {  // analytically impossible after a rejection; rounding can produce it
      *empty = true;
      k = icdf(vals, cnt, r64(x), margin);
      if (k < 0) k = 0;
    }
    *tok = ids[k];
    *prob = vals[k];
  };

  if (c.diag && !draft_all && (c.diag->pot_residual || c.diag->residual_margin)) {
    for (int32_t i = 0; i < L; ++i) {
      int32_t tok; float pr, mg; bool em;
      residual_at(i, &tok, &pr, &mg, &em);
      if (c.diag->pot_residual) c.diag->pot_residual[base + i] = tok;
      if (c.diag->residual_margin) c.diag->residual_margin[base + i] = mg;
    }
  }

  // Step 4: everything from the first failed test on is rejected
  int32_t a = draft_all ? 0 : orc_first_reject(ok.data(), L);
  c.out_accept_len[b] = a;

  for (int32_t i = 0; i < W; ++i) {
    const size_t r = base + i;
    int32_t tok = -1, flag = ORC_OUT_INVALID;
    float pr = 0.f;
    if (i < L) {
      if (draft_all) {
        tok = redraft_tok[(size_t)i]; pr = redraft_p[(size_t)i]; flag = ORC_OUT_RESAMPLED;
      } else if (i < a) {
        tok = c.drafts[r]; pr = ptok[(size_t)i]; flag = ORC_OUT_ACCEPTED;
      } else if (i == a) {
        float mg; bool em;
        residual_at(i, &tok, &pr, &mg, &em);
        if (em) st |= ORC_STATUS_EMPTY_RESIDUAL;
        flag = ORC_OUT_RESIDUAL;
      } else if (reuse[(size_t)i]) {
        tok = c.drafts[r]; pr = ptok[(size_t)i]; flag = ORC_OUT_REUSED;
      } else {
        tok = redraft_tok[(size_t)i]; pr = redraft_p[(size_t)i]; flag = ORC_OUT_RESAMPLED;
      }
    }
    c.out_tokens[r] = tok;
    c.out->tok_prob[r] = pr;
    if (c.out_flags) c.out_flags[r] = flag;
  }
  if (c.status) c.status[b] = st;
}

}  // namespace

extern "C" {

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) { philox(ctr, key, out); }

float orc_half_to_float(uint16_t bits) { return half_to_float(bits); }

float orc_uniform24(uint32_t x) { return uniform24(x); }

int32_t orc_row_probs(const void* cond, const void* uncond, int32_t dtype, int32_t V, float cfg_scale,
                      float inv_temperature, int32_t top_k, int32_t* ids, float* vals, int32_t* degenerate) {
  if (!cond || !ids || !vals) return -1;
  return row_probs(cond, uncond, dtype, 0, V, cfg_scale, inv_temperature, top_k, ids, vals, degenerate);
}

int32_t orc_accept(float p_tok, float q_tok, float u, float* ratio_out) { return accept(p_tok, q_tok, u, ratio_out); }

int32_t orc_first_reject(const int32_t* ok, int32_t L) {
  for (int32_t i = 0; i < L; ++i)
    if (!ok[i]) return i;
  return L;
}

int32_t orc_icdf(const float* w, int32_t n, uint64_t R, float* margin_out) { return icdf(w, n, R, margin_out); }

void orc_residual_weights(const int32_t* p_ids, const float* p_vals, int32_t p_cnt, const int32_t* q_ids,
                          const float* q_vals, int32_t q_cnt, int32_t V, float* w) {
  residual_weights(p_ids, p_vals, p_cnt, q_ids, q_vals, q_cnt, V, w);
}

int32_t orc_sjd_step(const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
                     const orc_probs* draft_probs, const orc_params* P, uint64_t philox_seed,
                     int32_t* out_accept_len, int32_t* out_tokens, orc_probs* out_probs, int32_t* out_flags,
                     int32_t* status, orc_diag* diag) {
  if (!P || !logits_cond || !out_accept_len || !out_tokens || !out_probs) return -1;
  if (!out_probs->tok_prob || !out_probs->ids || !out_probs->vals || !out_probs->cnt) return -1;
  if (P->B < 0 || P->W < 1 || P->V < 1 || P->top_k < 1) return -2;
  if (P->logits_dtype != ORC_F32 && P->logits_dtype != ORC_BF16 && P->logits_dtype != ORC_F16) return -3;
  const bool draft_all = (P->flags & ORC_FLAG_DRAFT_ALL) != 0;
  if (!draft_all) {
    if (!drafts || !draft_probs) return -1;
    if (!draft_probs->tok_prob || !draft_probs->ids || !draft_probs->vals || !draft_probs->cnt) return -1;
  }
  StepCtx c{logits_cond, logits_uncond, drafts, draft_probs, P, philox_seed, out_accept_len, out_tokens,
            out_probs, out_flags, status, diag, std::min(P->top_k, P->V)};
  const int64_t rows = (int64_t)P->B * P->W;
  std::vector<int32_t> degen((size_t)rows, 0);
  const int nt = std::max(1, P->n_threads);
  if (nt == 1) {
    rows_phase(c, 0, rows, &degen);
    for (int32_t b = 0; b < P->B; ++b) verify_phase(c, b, degen);
  } else {
    std::vector<std::thread> th;
    for (int t = 0; t < nt; ++t)
      th.emplace_back([&, t] { rows_phase(c, rows * t / nt, rows * (t + 1) / nt, &degen); });
    for (auto& x : th) x.join();
    th.clear();
    for (int t = 0; t < nt; ++t)
      th.emplace_back([&, t] {
        for (int32_t b = (int32_t)((int64_t)P->B * t / nt); b < (int32_t)((int64_t)P->B * (t + 1) / nt); ++b)
          verify_phase(c, b, degen);
      });
    for (auto& x : th) x.join();
  }
  return 0;
}

}  // extern "C"

// Verification stage of the step (paper Section 4.1, Steps 3 and 4): the accept test of Eq. acc-sjdpp
// on every row, the first-rejection prefix, the residual draw of Eq. rej-sjd at the first rejected row,
// and the reuse-or-redraw rule of Eq. reuse (Eq. refine-sjd when reuse is off) for the rows after it.
// One CTA per sequence; it reads what the row stage left in RowScratch and in out_probs.
#pragma once

#include "device_utils.cuh"
#include "row_kernels.cuh"

namespace sjd {

constexpr int kFlagReuse = 1;
constexpr int kFlagDraftAll = 2;
constexpr int kQUniform = -1;

constexpr int kOutInvalid = 0, kOutAccepted = 1, kOutResidual = 2, kOutReused = 3, kOutResampled = 4;
constexpr int kStatusQtok = 1, kStatusEmptyResidual = 2, kStatusDegenerate = 4, kStatusTimeout = 8;

struct VerifyArgs {
  int B, W, V, kcap;
  int flags;
  float tau;
  const int32_t* win_len;
  const int32_t* pos_base;
  const int32_t* iteration;
  int iteration0;
  int seq_base;
  uint32_t seed_lo, seed_hi;
  const int32_t* drafts;
  // previous-iteration distributions
  const float* q_tok;
  const int32_t* q_ids;
  const float* q_vals;
  const int32_t* q_cnt;
  // this call's distributions (written by the row stage)
  const int32_t* p_ids;
  const float* p_vals;
  const RowScratch* scratch;
  // outputs
  int32_t* out_accept_len;
  int32_t* out_tokens;
  float* out_tok_prob;
  int32_t* out_flags;
  int32_t* status;
};

// q(token) on a sparse row with ascending ids.
__device__ __forceinline__ float sparse_lookup(const int32_t* __restrict__ ids, const float* __restrict__ vals,
                                               int cnt, int token) {
  int lo = 0, hi = cnt;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (ids[mid] < token) lo = mid + 1;
    else hi = mid;
  }
  return (lo < cnt && ids[lo] == token) ? vals[lo] : 0.0f;
}

// ratio p/q of Eq. acc-sjdpp and of the confidence C (the same quantity), with the conventions for
// the corner cases: p == 0 gives 0 (never accepted, never reused); q <= 0 with p > 0 gives +inf.
__device__ __forceinline__ float likelihood_ratio(float p, float q) {
  if (p == 0.0f) return 0.0f;
  if (!(q > 0.0f)) return __int_as_float(0x7f800000);
  return __fdiv_rn(p, q);
}

struct VerifySmem {
  uint64_t scan[2 * 32 + 8];
  int first_reject;
  int status;
  int res_tok;
  float res_prob;
};

// Everything the verification stage does for sequence b, executed by NT threads (ranks `tid`).
template <int NT, int BAR>
__device__ void verify_sequence(const VerifyArgs& a, int b, int tid, VerifySmem& sm) {
  const int W = a.W;
  const int L = a.win_len ? min(max(a.win_len[b], 0), W) : W;
  const int pos0 = a.pos_base ? a.pos_base[b] : 0;
  const int iter = a.iteration ? a.iteration[b] : a.iteration0;
  const bool draft_all = (a.flags & kFlagDraftAll) != 0;
  const bool reuse_on = (a.flags & kFlagReuse) != 0;
  const size_t base = (size_t)b * W;
  if (tid == 0) {
    sm.first_reject = L;
    sm.status = 0;
    sm.res_tok = -1;
    sm.res_prob = 0.0f;
  }
  group_sync<NT, BAR>();

  // Step 3: r < min(1, p(x_i)/q(x_i)) on every valid row; the counter-based generator makes the
  // rows independent, so they are all tested at once
  for (int i = tid; i < L; i += NT) {
    const RowScratch rs = a.scratch[base + i];
    int st = (rs.status & kRowStatusDegenerate) ? kStatusDegenerate : 0;
    if (rs.status & kRowStatusTimeout) st |= kStatusTimeout;
    if (!draft_all) {
      const float q = a.q_tok[base + i];
      const float ratio = likelihood_ratio(rs.p_tok, q);
      const Philox4 rnd = philox4x32_10((uint32_t)(pos0 + i), (uint32_t)(a.seq_base + b), (uint32_t)iter, kPurposeAccept, a.seed_lo,
                                        a.seed_hi);
      const float u = uniform24(rnd.x0);
      if (!(u < fminf(ratio, 1.0f))) atomicMin(&sm.first_reject, i);
      if (!(q > 0.0f)) st |= kStatusQtok;
    }
    if (st) atomicOr(&sm.status, st);
  }
  group_sync<NT, BAR>();
  const int acc = draft_all ? 0 : sm.first_reject;

  // Step 4, first rejected row: draw from max(0, p - q) / sum max(0, p - q)
  if (!draft_all && acc < L) {
    const size_t r = base + acc;
    const int32_t* pid = a.p_ids + r * a.kcap;
    const float* pv = a.p_vals + r * a.kcap;
    const int32_t* qid = a.q_ids + r * a.kcap;
    const float* qv = a.q_vals + r * a.kcap;
    const int qc = a.q_cnt[r];
    const float q_uniform = __fdiv_rn(1.0f, (float)a.V);
    const Philox4 rnd = philox4x32_10((uint32_t)(pos0 + acc), (uint32_t)(a.seq_base + b), (uint32_t)iter, kPurposeResidual,
                                      a.seed_lo, a.seed_hi);
    auto residual = [&](int k) {
      const float q = (qc == kQUniform) ? q_uniform : sparse_lookup(qid, qv, qc, pid[k]);
      return fixed_weight(__fsub_rn(pv[k], q));
    };
    int k = group_icdf<NT, BAR>(residual, a.kcap, random64(rnd), tid, sm.scan);
    if (k < 0) {  // no mass left after rounding: draw from p itself
      if (tid == 0) sm.status |= kStatusEmptyResidual;
      k = group_icdf<NT, BAR>([&](int kk) { return fixed_weight(pv[kk]); }, a.kcap, random64(rnd), tid, sm.scan);
      if (k < 0) k = 0;
    }
    if (tid == 0) {
      sm.res_tok = pid[k];
      sm.res_prob = pv[k];
    }
  }
  group_sync<NT, BAR>();

  // Step 4, remaining rows, and the outputs
  for (int i = tid; i < W; i += NT) {
    int tok = -1, flag = kOutInvalid;
    float pr = 0.0f;
    if (i < L) {
      const RowScratch rs = a.scratch[base + i];
      if (draft_all) {
        tok = rs.samp_tok; pr = rs.samp_prob; flag = kOutResampled;
      } else if (i < acc) {
        tok = a.drafts[base + i]; pr = rs.p_tok; flag = kOutAccepted;
      } else if (i == acc) {
        tok = sm.res_tok; pr = sm.res_prob; flag = kOutResidual;
      } else {
        const float C = likelihood_ratio(rs.p_tok, a.q_tok[base + i]);  // confidence of Eq. (C)
        if (reuse_on && rs.p_tok > 0.0f && C > a.tau) {
          tok = a.drafts[base + i]; pr = rs.p_tok; flag = kOutReused;
        } else {
          tok = rs.samp_tok; pr = rs.samp_prob; flag = kOutResampled;
        }
      }
    }
    a.out_tokens[base + i] = tok;
    a.out_tok_prob[base + i] = pr;
    if (a.out_flags) a.out_flags[base + i] = flag;
  }
  if (tid == 0) {
    a.out_accept_len[b] = acc;
    if (a.status) a.status[b] = sm.status;
  }
  group_sync<NT, BAR>();
}

template <int NT>
__global__ void __launch_bounds__(NT) verify_kernel(const VerifyArgs a) {
  __shared__ VerifySmem sm;
  for (int b = blockIdx.x; b < a.B; b += gridDim.x) verify_sequence<NT, 0>(a, b, threadIdx.x, sm);
}

}  // namespace sjd

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
constexpr int kStatusQtok = 1, kStatusEmptyResidual = 2, kStatusDegenerate = 4, kStatusTimeout = 8, kStatusRedone = 16;

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

constexpr int kVerifyStageCap = 2048;  // entries of a previous-iteration row staged in shared memory

struct VerifySmem {
  uint64_t scan[2 * 32 + 8];
  int32_t q_ids[kVerifyStageCap];
  float q_vals[kVerifyStageCap];
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
  int flip = 0;
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
    if (rs.status & kRowStatusRedone) st |= kStatusRedone;
    if (!draft_all) {
      const float q = a.q_tok[base + i];
      const float ratio = likelihood_ratio(rs.p_tok, q);
      const Philox4 rnd = philox4x32_10((uint32_t)(pos0 + i), (uint32_t)(a.seq_base + b), (uint32_t)iter, kPurposeAccept,
                                        a.seed_lo, a.seed_hi);
      const float u = uniform24(rnd.x0);
      if (!(u < fminf(ratio, 1.0f))) atomicMin(&sm.first_reject, i);
      if (!(q > 0.0f)) st |= kStatusQtok;
    }
    if (st) atomicOr(&sm.status, st);
  }
  group_sync<NT, BAR>();
  const int acc = draft_all ? 0 : sm.first_reject;

  // Step 4, first rejected row: draw from max(0, p - q) / sum max(0, p - q).  Every thread owns a run of
  // consecutive entries of p_a (ascending token id), so one scan of the per-thread sums locates the draw.
  if (!draft_all && acc < L) {
    const size_t r = base + acc;
    const int kcap = a.kcap;
    const int32_t* pid = a.p_ids + r * kcap;
    const float* pv = a.p_vals + r * kcap;
    const int32_t* qid = a.q_ids + r * kcap;
    const float* qv = a.q_vals + r * kcap;
    const int qc = a.q_cnt[r];
    const bool staged = qc > 0 && qc <= kVerifyStageCap;
    if (staged) {
      for (int k = tid; k < qc; k += NT) {
        sm.q_ids[k] = qid[k];
        sm.q_vals[k] = qv[k];
      }
      group_sync<NT, BAR>();
    }
    const int32_t* sid = staged ? sm.q_ids : qid;
    const float* sval = staged ? sm.q_vals : qv;
    const float q_uniform = __fdiv_rn(1.0f, (float)a.V);
    const Philox4 rnd = philox4x32_10((uint32_t)(pos0 + acc), (uint32_t)(a.seq_base + b), (uint32_t)iter,
                                      kPurposeResidual, a.seed_lo, a.seed_hi);
    const uint64_t R = random64(rnd);
    const int per = (kcap + NT - 1) / NT;
    const int k0 = min(tid * per, kcap), k1 = min(k0 + per, kcap);
    int found = -1;
    for (int attempt = 0; attempt < 2; ++attempt) {
      // attempt 0: residual weights; attempt 1 (only when they sum to zero after rounding): p itself
      uint64_t local = 0;
      for (int k = k0; k < k1; ++k) {
        float w = pv[k];
        if (attempt == 0) {
          const float q = (qc == kQUniform) ? q_uniform : sparse_lookup(sid, sval, max(qc, 0), pid[k]);
          w = __fsub_rn(w, q);
        }
        local += fixed_weight(w);
      }
      uint64_t T;
      const uint64_t lo = group_scan1<NT, BAR, uint64_t>(local, tid, sm.scan, flip, &T);
      if (T == 0) {
        if (attempt == 0) {
          if (tid == 0) sm.status |= kStatusEmptyResidual;
          continue;
        }
        if (tid == 0) found = 0;
        break;
      }
      const uint64_t t = __umul64hi(R, T);
      if (t >= lo && t < lo + local) {
        uint64_t run = lo;
        for (int k = k0; k < k1; ++k) {
          float w = pv[k];
          if (attempt == 0) {
            const float q = (qc == kQUniform) ? q_uniform : sparse_lookup(sid, sval, max(qc, 0), pid[k]);
            w = __fsub_rn(w, q);
          }
          run += fixed_weight(w);
          if (t < run) {
            found = k;
            break;
          }
        }
      }
      break;
    }
    if (found >= 0) {
      sm.res_tok = pid[found];
      sm.res_prob = pv[found];
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
  // Launched with programmatic stream serialisation right behind the row kernel: the grid may be scheduled
  // while that kernel's last rows are still running, and waits here until all of its writes are visible.
  // A no-op after an ordinary launch.
  grid_dependency_wait();
  // a following kernel that waits the same way (the next step's row kernel) may set itself up meanwhile
  allow_dependent_launch();
  for (int b = blockIdx.x; b < a.B; b += gridDim.x) verify_sequence<NT, 0>(a, b, threadIdx.x, sm);
}

}  // namespace sjd

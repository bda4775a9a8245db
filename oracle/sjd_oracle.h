/*
 * CPU oracle for one speculative-Jacobi verify-and-redraft step (SJD / SJD++).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, single-file
 * C++ restatement of the paper's definitions (Section 3.1 sampling head, Section 4.1
 * Steps 3-4, Eq. acc-sjdpp, Eq. rej-sjd, the confidence ratio C and Eq. reuse, and
 * Eq. refine-sjd for plain SJD).  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code, header, table or
 * constant generator with the CUDA library and neither includes the other.
 *
 * Every pointer in this header is a HOST pointer.  Probabilities are computed in
 * double precision and rounded once to float; every decision that turns a float into
 * an integer (accept test, reuse test, fixed-point weights of the sampler) is then
 * taken on those floats with individually rounded fp32 operations, which is the
 * precision the CUDA path decides in.
 *
 * Parity status of each part ("pinned" = checked by the CPU tests against something
 * other than this file):
 *   philox4x32-10 ............ pinned (published known-answer vectors, uniformity)
 *   row distribution ......... pinned (fp64 library softmax/top-k, exact small cases)
 *   accept test .............. pinned (closed forms of the appendix proof, 1e6 trials)
 *   first-rejection prefix ... pinned (brute force over all masks)
 *   integer inverse CDF ...... pinned (exhaustive sweep of t, permutation invariance)
 *   residual resampling ...... pinned (closed forms, exact marginal preservation)
 *   reuse / redraft .......... pinned (invariants, special cases tau = +-inf, K = 1)
 *   decode loop .............. pinned by invariants only beyond the step it calls
 */
#ifndef SJD_ORACLE_H_
#define SJD_ORACLE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_F16 = 2 };

/* flags */
enum {
  ORC_FLAG_REUSE = 1,     /* SJD++ confidence reuse (Eq. reuse); off = plain SJD (Eq. refine-sjd) */
  ORC_FLAG_DRAFT_ALL = 2  /* no verification: every valid row is sampled from its own p (initial draft) */
};

/* Philox counter word 3: what the random number is used for */
enum { ORC_PURPOSE_ACCEPT = 0, ORC_PURPOSE_RESIDUAL = 1, ORC_PURPOSE_REDRAFT = 2, ORC_PURPOSE_INIT = 3 };

/* per-position outcome written to out_flags */
enum { ORC_OUT_INVALID = 0, ORC_OUT_ACCEPTED = 1, ORC_OUT_RESIDUAL = 2, ORC_OUT_REUSED = 3, ORC_OUT_RESAMPLED = 4 };

/* per-sequence status bits */
enum {
  ORC_STATUS_QTOK_NONPOSITIVE = 1, /* a valid row had q(x_i) <= 0 */
  ORC_STATUS_EMPTY_RESIDUAL = 2,   /* fixed-point residual total was 0; sampled from p instead */
  ORC_STATUS_DEGENERATE_ROW = 4    /* a row had no finite logit: all probabilities 0 */
};

#define ORC_Q_UNIFORM (-1) /* cnt value: the row is the uniform distribution over V, 1/V each */

typedef struct {
  float* tok_prob; /* [B,W]      probability of the token in the matching token array */
  int32_t* ids;    /* [B,W,kcap] support, ascending token id                          */
  float* vals;     /* [B,W,kcap] probability on that support                          */
  int32_t* cnt;    /* [B,W]      entries used, or ORC_Q_UNIFORM                       */
} orc_probs;

typedef struct {
  int32_t B, W, V;
  int32_t logits_dtype;       /* ORC_F32 / ORC_BF16 / ORC_F16 (raw 16-bit patterns)            */
  int64_t stride_b, stride_w; /* element strides of both logits arrays; vocabulary contiguous  */
  float cfg_scale;            /* s of the guidance merge                                       */
  float inv_temperature;      /* 1/T, already rounded to float by the caller                   */
  int32_t top_k;              /* kcap = min(top_k, V)                                          */
  float reuse_tau;
  int32_t flags;
  const int32_t* win_len;   /* [B] valid rows per sequence, NULL = W                          */
  const int32_t* pos_base;  /* [B] absolute position of window row 0, NULL = 0                */
  const int32_t* iteration; /* [B] Jacobi iteration index, NULL = iteration0                  */
  int32_t iteration0;
  int32_t n_threads;        /* rows are split over this many std::thread workers (>=1)        */
  int32_t seq_base;         /* global index of sequence 0 of this call: the Philox counter's
                               sequence word is seq_base + b (a batch split over several
                               calls or devices draws the same numbers as the whole batch)   */
} orc_params;

/* Optional per-position diagnostics (any pointer may be NULL).  "Potential" outcomes are
 * evaluated for EVERY valid row as if that row were in the corresponding role, which lets a
 * test follow either branch of a decision whose margin is below the comparison threshold. */
typedef struct {
  float* u;               /* [B,W] uniform drawn for the accept test                              */
  float* ratio;           /* [B,W] p(x_i)/q(x_i) as used by the accept and reuse tests            */
  float* accept_margin;   /* [B,W] |u - ratio|                                                    */
  float* reuse_margin;    /* [B,W] |ratio - tau|                                                  */
  int32_t* pot_ok;        /* [B,W] accept decision of the row                                     */
  int32_t* pot_reuse;     /* [B,W] reuse decision of the row (flags and tau applied)              */
  int32_t* pot_redraft;   /* [B,W] token the row gets if it is resampled from p                   */
  float* redraft_margin;  /* [B,W] distance of t to the nearest CDF step, in probability mass     */
  int32_t* pot_residual;  /* [B,W] token the row gets if it is the first rejected row             */
  float* residual_margin; /* [B,W] same distance for the residual sampler                         */
} orc_diag;

/* Philox4x32-10 block function (Salmon et al., SC'11). */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* u = (x >> 8) * 2^-24, in [0,1). */
float orc_uniform24(uint32_t x);

/* Value of an IEEE 754 binary16 pattern, widened exactly to fp32 (the storage type of fp16 logits). */
float orc_half_to_float(uint16_t bits);

/* Sampling head for one row (Section 3.1; guidance weight and top-K of Section 5.1):
 * merged = uncond + s*(cond - uncond); y = merged / T; keep the kcap largest y (ties to the lower
 * id); softmax over the survivors.  Writes kcap ids (ascending) and kcap probabilities, returns
 * kcap, or -1 on bad arguments.  uncond may be NULL (no guidance).  *degenerate is set to 1 when no
 * logit is finite. */
int32_t orc_row_probs(const void* cond, const void* uncond, int32_t dtype, int32_t V, float cfg_scale,
                      float inv_temperature, int32_t top_k, int32_t* ids, float* vals, int32_t* degenerate);

/* Accept test of Eq. acc-sjdpp on float probabilities: 1 = accept. */
int32_t orc_accept(float p_tok, float q_tok, float u, float* ratio_out);

/* First index whose flag is 0, or L when all are set (Step 4, "remaining tokens are rejected"). */
int32_t orc_first_reject(const int32_t* ok, int32_t L);

/* Fixed-point inverse CDF: W_k = floor(w_k * 2^40); T = sum W_k; t = floor(R*T / 2^64);
 * returns the smallest k with W_0+..+W_k > t, or -1 when T == 0.  margin_out (optional) receives
 * min(t - P_{k-1}, P_k - t) / 2^40, the distance of t to the nearest step of the CDF in units of
 * probability mass (P_k = W_0+..+W_k). */
int32_t orc_icdf(const float* w, int32_t n, uint64_t R, float* margin_out);

/* Residual weights of Eq. rej-sjd on a sparse p row against a sparse (or uniform) q row:
 * w_k = max(0, p_vals[k] - q(p_ids[k])) in fp32. */
void orc_residual_weights(const int32_t* p_ids, const float* p_vals, int32_t p_cnt, const int32_t* q_ids,
                          const float* q_vals, int32_t q_cnt, int32_t V, float* w);

/* One verify-and-redraft step for B sequences (Section 4.1, Steps 3 and 4).  Returns 0, or a
 * negative value for bad arguments.  out_flags, status and diag may be NULL.  logits_uncond may be
 * NULL.  drafts and draft_probs may be NULL when ORC_FLAG_DRAFT_ALL is set. */
int32_t orc_sjd_step(const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
                     const orc_probs* draft_probs, const orc_params* params, uint64_t philox_seed,
                     int32_t* out_accept_len, int32_t* out_tokens, orc_probs* out_probs, int32_t* out_flags,
                     int32_t* status, orc_diag* diag);

#ifdef __cplusplus
}
#endif
#endif

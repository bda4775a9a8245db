// Window bookkeeping between two Jacobi iterations (paper Section 4.1, Step 1 and the closing sentence of
// Step 4): the accepted prefix and the residual token are committed, the rows that remain unaccepted move
// to the front of the window and keep this iteration's distributions as their verification reference,
// and the freed slots are filled with newly initialised tokens: random ones whose reference distribution
// is uniform (Section 4.2's baseline), or one of the four spatial-prior strategies of Section 4.2 - the
// token of the left or above neighbour on the raster grid (a deterministic draft: point-mass reference),
// or a draw from the prediction the step just made for that neighbour (that prediction is the reference).
#pragma once

#include "device_utils.cuh"

namespace sjd {

constexpr int kPurposeTokenInit = 4;  // Philox purpose of a randomly initialised draft token
constexpr int kPurposePriorInit = 5;  // Philox purpose of a draft drawn from a neighbour's prediction

constexpr int kInitRandom = 0, kInitRepeatLeft = 1, kInitRepeatAbove = 2, kInitSampleLeft = 3, kInitSampleAbove = 4;

struct AdvanceArgs {
  int B, W, V, kcap, n_total;
  int seq_base;
  int init_mode, grid_width;
  int no_refine;  // 1: nothing is carried over, every slot behind the committed tokens is newly initialised
  uint32_t seed_lo, seed_hi;
  // result of the step that just ran
  const int32_t* accept_len;
  const int32_t* step_tokens;
  const float* step_tok_prob;
  const int32_t* step_ids;
  const float* step_vals;
  const int32_t* step_cnt;
  // window state (read here, updated by advance_state_kernel)
  int32_t* win_len;
  int32_t* pos_base;
  int32_t* iteration;
  // next iteration's drafts and their reference distributions
  int32_t* next_drafts;
  float* next_tok_prob;
  int32_t* next_ids;
  float* next_vals;
  int32_t* next_cnt;
  // committed tokens, [B, n_total]
  int32_t* committed;
  int32_t* n_committed;  // [B] optional: tokens committed by this call
};

// Tokens committed by a step: the accepted prefix plus the residual draw at the first rejected row, or
// the whole window when every row was accepted.
__device__ __forceinline__ int commit_count(int a, int L) { return a < L ? a + 1 : L; }

// A token drawn uniformly from [0, V) for absolute position `pos`: floor(x0 * V / 2^32).
__device__ __forceinline__ int random_token(int pos, int seq, int iter, int V, uint32_t k0, uint32_t k1) {
  const Philox4 r = philox4x32_10((uint32_t)pos, (uint32_t)seq, (uint32_t)iter, kPurposeTokenInit, k0, k1);
  return (int)(((uint64_t)r.x0 * (uint64_t)(uint32_t)V) >> 32);
}

// One block per (sequence, next-window row).
template <int NT>
__global__ void __launch_bounds__(NT) advance_rows_kernel(const AdvanceArgs a) {
  // launched as a programmatic dependent of the step's verification kernel: wait for its results, then
  // let the kernel behind this one be placed early in turn
  grid_dependency_wait();
  allow_dependent_launch();
  const int b = blockIdx.x / a.W, i = blockIdx.x - b * a.W;
  const int L = min(max(a.win_len[b], 0), a.W);
  const int pos0 = a.pos_base[b];
  const int iter = a.iteration[b];
  const int acc = min(max(a.accept_len[b], 0), L);
  const int c = commit_count(acc, L);
  const int pos1 = pos0 + c;
  const int L1 = max(0, min(a.W, a.n_total - pos1));
  const size_t row = (size_t)b * a.W + i;
  // commit: rows 0..c-1 of this step's tokens
  if (i < c && threadIdx.x == 0 && pos0 + i < a.n_total) a.committed[(size_t)b * a.n_total + pos0 + i] = a.step_tokens[row];
  int32_t* nid = a.next_ids + row * a.kcap;
  float* nv = a.next_vals + row * a.kcap;
  if (i >= L1) {
    if (threadIdx.x == 0) {
      a.next_drafts[row] = -1;
      a.next_tok_prob[row] = 0.0f;
      a.next_cnt[row] = 0;
    }
    return;
  }
  const int src = i + c;
  if (!a.no_refine && src < L) {
    // an unaccepted row moves up; its distribution of this iteration becomes the reference
    const size_t srow = (size_t)b * a.W + src;
    const int32_t* sid = a.step_ids + srow * a.kcap;
    const float* sv = a.step_vals + srow * a.kcap;
    const int n = a.step_cnt[srow];
    for (int k = threadIdx.x; k < n; k += NT) {
      nid[k] = sid[k];
      nv[k] = sv[k];
    }
    if (threadIdx.x == 0) {
      a.next_drafts[row] = a.step_tokens[srow];
      a.next_tok_prob[row] = a.step_tok_prob[srow];
      a.next_cnt[row] = n;
    }
    return;
  }
  // a new slot at absolute position p
  const int p = pos1 + i;
  const int G = a.grid_width;
  const int pred_end = pos0 + L;                      // first position the step made no prediction for
  const int tok_end = a.no_refine ? pos1 : pred_end;  // first position whose token does not survive the step
  const int mode = a.init_mode;
  const bool above = (mode == kInitRepeatAbove || mode == kInitSampleAbove) && p >= G;
  const bool sample = mode == kInitSampleLeft || mode == kInitSampleAbove;
  if (mode == kInitRandom || L < 1) {
    if (threadIdx.x == 0) {
      a.next_drafts[row] = random_token(p, a.seq_base + b, iter, a.V, a.seed_lo, a.seed_hi);
      a.next_tok_prob[row] = __fdiv_rn(1.0f, (float)a.V);
      a.next_cnt[row] = -1;
    }
    return;
  }
  // the position whose token (repeat) or prediction (sample) initialises this slot
  int r;
  if (!sample) {
    // positions at or after tok_end are new slots themselves: follow their own rule back into known tokens
    r = above ? p - G : p - 1;
    while (r >= tok_end) r -= (mode == kInitRepeatAbove && r >= G) ? G : 1;
  } else {
    const int left = min(p - 1, pred_end - 1);  // the prediction made for p-1, else the last one made
    if (above) {
      r = p - G;
      while (r >= pred_end) r -= G;
      if (r < 0) r = left;  // left the grid: as for "sample left"
    } else {
      r = left;
    }
  }
  if (!sample || r < pos0) {
    if (threadIdx.x == 0) {
      const int tok = r < pos0 ? a.committed[(size_t)b * a.n_total + r] : a.step_tokens[(size_t)b * a.W + (r - pos0)];
      a.next_drafts[row] = tok;
      a.next_tok_prob[row] = 1.0f;
      nid[0] = tok;
      nv[0] = 1.0f;
      a.next_cnt[row] = 1;
    }
    return;
  }
  // draw from the prediction of row r - pos0 and keep that prediction as the reference
  __shared__ uint64_t scratch[2 * (NT / 32) + 4];
  const size_t srow = (size_t)b * a.W + (r - pos0);
  const int32_t* sid = a.step_ids + srow * a.kcap;
  const float* sv = a.step_vals + srow * a.kcap;
  const int n = min(max(a.step_cnt[srow], 0), a.kcap);
  for (int k = threadIdx.x; k < n; k += NT) {
    nid[k] = sid[k];
    nv[k] = sv[k];
  }
  const Philox4 rnd = philox4x32_10((uint32_t)p, (uint32_t)(a.seq_base + b), (uint32_t)iter, kPurposePriorInit,
                                    a.seed_lo, a.seed_hi);
  int k = group_icdf<NT, 0>([&](int j) { return fixed_weight(sv[j]); }, n, random64(rnd), threadIdx.x, scratch);
  if (k < 0) k = 0;
  if (threadIdx.x == 0) {
    a.next_drafts[row] = n > 0 ? sid[k] : 0;
    a.next_tok_prob[row] = n > 0 ? sv[k] : 0.0f;
    a.next_cnt[row] = n;
  }
}

// One thread per sequence: the window state after the commit.  Runs after advance_rows_kernel.
__global__ void advance_state_kernel(const AdvanceArgs a) {
  grid_dependency_wait();  // advance_rows_kernel reads the state this kernel overwrites
  allow_dependent_launch();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= a.B) return;
  const int L = min(max(a.win_len[b], 0), a.W);
  const int acc = min(max(a.accept_len[b], 0), L);
  const int c = commit_count(acc, L);
  const int pos1 = a.pos_base[b] + c;
  a.pos_base[b] = pos1;
  a.win_len[b] = max(0, min(a.W, a.n_total - pos1));
  a.iteration[b] = a.iteration[b] + 1;
  if (a.n_committed) a.n_committed[b] = c;
}

// First window of a sequence.  With a spatial-prior strategy slot i copies slot i-1 (the "left" strategies,
// and the "above" ones in the first grid row) or slot i-G; either way the chain ends at slot 0, whose
// token is random, so every slot holds that token.  No prediction exists yet, so the sampling strategies
// repeat as well.  With the random strategy every slot gets its own uniform token.
__global__ void init_window_kernel(const AdvanceArgs a) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= a.B * a.W) return;
  const int b = r / a.W, i = r - b * a.W;
  const int L = min(max(a.win_len[b], 0), a.W);
  if (i >= L) {
    a.next_drafts[r] = -1;
    a.next_tok_prob[r] = 0.0f;
    a.next_cnt[r] = 0;
    return;
  }
  const int src = a.init_mode == kInitRandom ? i : 0;
  const int tok = random_token(a.pos_base[b] + src, a.seq_base + b, a.iteration[b], a.V, a.seed_lo, a.seed_hi);
  a.next_drafts[r] = tok;
  if (a.init_mode == kInitRandom || i == 0) {
    a.next_tok_prob[r] = __fdiv_rn(1.0f, (float)a.V);
    a.next_cnt[r] = -1;
  } else {
    a.next_tok_prob[r] = 1.0f;
    a.next_ids[(size_t)r * a.kcap] = tok;
    a.next_vals[(size_t)r * a.kcap] = 1.0f;
    a.next_cnt[r] = 1;
  }
}

}  // namespace sjd

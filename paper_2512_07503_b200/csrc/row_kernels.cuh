// Sampling head of the step (paper Section 3.1): guidance merge, temperature, top-K, softmax over the
// survivors, plus the per-row draw every row may need later (Eq. reuse second case / Eq. refine-sjd).
//
// `row_generic` is the any-shape path: it works through global memory only (the row stays in L2 after
// its first read), has no capacity limit on K or V, and is also what the streaming kernel falls back
// to for a row it cannot finish on chip.
#pragma once

#include "device_utils.cuh"

namespace sjd {

// What the row stage leaves for the verification stage, one record per window row.
struct RowScratch {
  float p_tok;       // p_i(x_i): probability of the draft token under this call's distribution
  int32_t samp_tok;  // token drawn from p_i with this row's redraft/init counter
  float samp_prob;   // p_i(samp_tok)
  int32_t status;    // kRowStatus* bits
};

struct RowArgs {
  const void* cond;
  const void* uncond;
  int64_t stride_b, stride_w;  // elements
  int B, W, V, kcap;
  float s, inv_T;
  const int32_t* win_len;
  const int32_t* pos_base;
  const int32_t* iteration;
  int iteration0;
  int seq_base;  // global index of sequence 0 (sequence word of the generator's counter)
  const int32_t* drafts;  // nullptr when every row is drafted
  uint32_t seed_lo, seed_hi;
  int purpose;  // kPurposeRedraft or kPurposeInit
  int32_t* out_ids;
  float* out_vals;
  int32_t* out_cnt;
  RowScratch* scratch;
};

struct GenericSmem {
  uint32_t hist[256];
  uint64_t scan[2 * 32 + 8];
  uint32_t sel_digit, sel_above;
  float p_tok;
};

__device__ __forceinline__ const void* row_ptr(const void* base, int dtype, int64_t elem) {
  return base == nullptr ? nullptr
                         : static_cast<const void*>(static_cast<const char*>(base) + elem * (dtype == 0 ? 4 : 2));
}

// One row through global memory.  All NT threads of the group call it with the same arguments.
template <int DTYPE, int NT, int BAR>
__device__ void row_generic(const RowArgs& a, int row, int tid, GenericSmem& sm, int extra_status = 0) {
  const int b = row / a.W, i = row - b * a.W;
  const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
  RowScratch* rs = a.scratch + row;
  if (i >= L) {
    if (tid == 0) {
      a.out_cnt[row] = 0;
      *rs = RowScratch{0.0f, -1, 0.0f, 0};
    }
    return;
  }
  const int V = a.V, kcap = a.kcap;
  const int64_t off = (int64_t)b * a.stride_b + (int64_t)i * a.stride_w;
  const void* cond = row_ptr(a.cond, DTYPE, off);
  const void* uncond = row_ptr(a.uncond, DTYPE, off);
  int32_t* ids = a.out_ids + (size_t)row * kcap;
  float* vals = a.out_vals + (size_t)row * kcap;

  // ---- exact key of the kcap-th largest y: MSB-first radix select, 8 bits per pass ----
  uint32_t prefix = 0, prefix_mask = 0, remaining = (uint32_t)kcap;
  float vmax = __int_as_float(0xff800000);
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int j = tid; j < 256; j += NT) sm.hist[j] = 0;
    group_sync<NT, BAR>();
    for (int e = tid * 8; e < V; e += NT * 8) {
      float y[8];
      load_y8<DTYPE>(cond, uncond, e, a.s, a.inv_T, y);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t k = float_key(y[j]);
        if (pass == 0) vmax = fmaxf(vmax, y[j]);
        if ((k & prefix_mask) == prefix) atomicAdd(&sm.hist[(k >> shift) & 0xffu], 1u);
      }
    }
    group_sync<NT, BAR>();
    if (tid < 32) {
      // lane l owns digits 255-8l .. 248-8l; walk from the largest digit down
      uint32_t c[8], sum = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        c[j] = sm.hist[255 - 8 * tid - j];
        sum += c[j];
      }
      uint32_t inc = sum;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, inc, d);
        if (tid >= d) inc += n;
      }
      uint32_t above = inc - sum;  // entries in digits larger than this lane's
      if (above < remaining && remaining <= inc) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (above < remaining && remaining <= above + c[j]) {
            sm.sel_digit = 255 - 8 * tid - j;
            sm.sel_above = above;
          }
          above += c[j];
        }
      }
    }
    group_sync<NT, BAR>();
    prefix |= sm.sel_digit << shift;
    prefix_mask |= 0xffu << shift;
    remaining -= sm.sel_above;
  }
  const uint32_t thr = prefix;        // key of the kcap-th largest value
  const uint32_t need = remaining;    // how many entries equal to it are kept (lowest ids)
  const float m = group_max_f32<NT, BAR>(vmax, tid, sm.scan);

  // ---- ordered compaction: ids ascending, y parked in vals ----
  uint32_t gt_base = 0, eq_base = 0;
  for (int c0 = 0; c0 < V; c0 += NT * 8) {
    const int e = c0 + tid * 8;
    float y[8];
    uint32_t gt = 0, eq = 0;
    if (e < V) {
      load_y8<DTYPE>(cond, uncond, e, a.s, a.inv_T, y);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t k = float_key(y[j]);
        gt |= (k > thr ? 1u : 0u) << j;
        eq |= (k == thr ? 1u : 0u) << j;
      }
    }
    uint32_t total;
    const uint32_t packed = (uint32_t)__popc(gt) | ((uint32_t)__popc(eq) << 16);
    const uint32_t ex = group_exclusive_scan<NT, BAR, uint32_t>(packed, tid, sm.scan, &total);
    const uint32_t gt_before = gt_base + (ex & 0xffffu), eq_before = eq_base + (ex >> 16);
    if (e < V) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t below = (1u << j) - 1u;
        const uint32_t g = gt_before + __popc(gt & below), q = eq_before + __popc(eq & below);
        const bool take = ((gt >> j) & 1u) || (((eq >> j) & 1u) && q < need);
        if (take) {
          const uint32_t pos = g + min(q, need);
          ids[pos] = e + j;
          vals[pos] = y[j];
        }
      }
    }
    gt_base += total & 0xffffu;
    eq_base += total >> 16;
  }
  group_sync<NT, BAR>();

  // ---- softmax over the survivors ----
  // no finite maximum (nothing finite in the row, or an infinite logit): all probabilities are reported as 0
  const bool degenerate = !(fabsf(m) <= 3.402823466e38f);
  float zpart = 0.0f;
  for (int k = tid; k < kcap; k += NT) {
    const float e = degenerate ? 0.0f : exp_diff(vals[k], m);
    vals[k] = e;
    zpart += e;
  }
  const float Z = group_sum_f32<NT, BAR>(zpart, tid, sm.scan);
  const int draft = a.drafts ? a.drafts[row] : -1;
  if (tid == 0) sm.p_tok = 0.0f;
  group_sync<NT, BAR>();
  for (int k = tid; k < kcap; k += NT) {
    const float p = degenerate ? 0.0f : __fdiv_rn(vals[k], Z);
    vals[k] = p;
    if (ids[k] == draft) sm.p_tok = p;
  }
  group_sync<NT, BAR>();

  // ---- the row's own draw from p_i ----
  const int pos = (a.pos_base ? a.pos_base[b] : 0) + i;
  const int iter = a.iteration ? a.iteration[b] : a.iteration0;
  const Philox4 rnd = philox4x32_10((uint32_t)pos, (uint32_t)(a.seq_base + b), (uint32_t)iter, (uint32_t)a.purpose, a.seed_lo,
                                    a.seed_hi);
  int k = group_icdf<NT, BAR>([&](int kk) { return fixed_weight(vals[kk]); }, kcap, random64(rnd), tid, sm.scan);
  if (k < 0) k = 0;
  if (tid == 0) {
    a.out_cnt[row] = kcap;
    *rs = RowScratch{sm.p_tok, ids[k], vals[k], (degenerate ? kRowStatusDegenerate : 0) | extra_status};
  }
  group_sync<NT, BAR>();
}

template <int DTYPE, int NT>
__global__ void __launch_bounds__(NT) rows_generic_kernel(const RowArgs a) {
  __shared__ GenericSmem sm;
  const int rows = a.B * a.W;
  grid_dependency_wait();  // a launch allowed to overlap the stream's previous kernel waits for its end here
  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    // from the block's last row on, the verification grid may be scheduled (it waits for this grid's end)
    if (row + (int)gridDim.x >= rows) allow_dependent_launch();
    row_generic<DTYPE, NT, 0>(a, row, threadIdx.x, sm);
  }
}

}  // namespace sjd

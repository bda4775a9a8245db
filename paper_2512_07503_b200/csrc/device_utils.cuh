// Device-side building blocks shared by the kernels of the step: Philox4x32-10, the order-preserving
// key of a float, logit loads with the guidance merge, and block-wide scans / reductions that work on
// any group of NT threads synchronised by a named barrier.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sjd {

constexpr int kPurposeAccept = 0;
constexpr int kPurposeResidual = 1;
constexpr int kPurposeRedraft = 2;
constexpr int kPurposeInit = 3;

constexpr int kRowStatusDegenerate = 1;
constexpr int kRowStatusTimeout = 2;  // a bounded on-chip wait gave up; the row has no result
constexpr int kRowStatusRedone = 4;   // the single-pass kernel handed the row to the any-shape path (result exact)

// ------------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): counter = (position, sequence, iteration, purpose),
// key = (seed low, seed high).
// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch: a kernel lets the next kernel of its stream be scheduled early
// (allow_dependent_launch), and that kernel blocks in grid_dependency_wait() until the first has completed
// and its memory operations are visible.
__device__ __forceinline__ void allow_dependent_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct Philox4 {
  uint32_t x0, x1, x2, x3;
};

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return Philox4{c0, c1, c2, c3};
}

__device__ __forceinline__ float uniform24(uint32_t x) { return (float)(x >> 8) * (1.0f / 16777216.0f); }

__device__ __forceinline__ uint64_t random64(const Philox4& p) { return (uint64_t)p.x0 | ((uint64_t)p.x1 << 32); }

// ------------------------------------------------------------------------------------------------
// Order-preserving map float -> uint32 (larger float <=> larger key); -0 is folded into +0 and NaN
// ranks with -inf before the key is taken.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float canonical(float y) {
  if (!(y == y)) return __int_as_float(0xff800000);  // NaN -> -inf
  return __fadd_rn(y, 0.0f);                         // -0 -> +0
}

__device__ __forceinline__ uint32_t float_key(float y) {
  const uint32_t b = __float_as_uint(y);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Guidance merge and temperature with one rounding per operation (the result decides the top-K set):
// d = c - u; g = fma(s, d, u); y = g * inv_T.
__device__ __forceinline__ float merge_logit(float c, float u, float s, float inv_T) {
  const float d = __fsub_rn(c, u);
  const float g = __fmaf_rn(s, d, u);
  return __fmul_rn(g, inv_T);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
// the two IEEE half-precision values of a 32-bit word, widened exactly
__device__ __forceinline__ float2 f16_pair(uint32_t w) { return __half22float2(*reinterpret_cast<const __half2*>(&w)); }

// Eight consecutive logits starting at element `e` (a multiple of 8) of a row, converted to fp32.
template <int DTYPE>
__device__ __forceinline__ void load8(const void* __restrict__ row, int e, float (&x)[8]) {
  if (DTYPE == 1) {
    const uint4 w = __ldg(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(row) + e));
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
  } else if (DTYPE == 2) {
    const uint4 w = __ldg(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(row) + e));
    const float2 a = f16_pair(w.x), b = f16_pair(w.y), c = f16_pair(w.z), d = f16_pair(w.w);
    x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y; x[4] = c.x; x[5] = c.y; x[6] = d.x; x[7] = d.y;
  } else {
    const float4 a = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(row) + e));
    const float4 b = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(row) + e) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  }
}

// y of eight consecutive vocabulary entries (canonical form).
template <int DTYPE>
__device__ __forceinline__ void load_y8(const void* __restrict__ cond, const void* __restrict__ uncond, int e, float s,
                                        float inv_T, float (&y)[8]) {
  float c[8];
  load8<DTYPE>(cond, e, c);
  if (uncond != nullptr) {
    float u[8];
    load8<DTYPE>(uncond, e, u);
#pragma unroll
    for (int j = 0; j < 8; ++j) y[j] = canonical(merge_logit(c[j], u[j], s, inv_T));
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) y[j] = canonical(__fmul_rn(c[j], inv_T));
  }
}

// exp(y - m) for y <= m with the rounding error of the fp32 subtraction compensated, so that the
// result is within a few ulp of the exact exponential of the exact difference.
__device__ __forceinline__ float exp_diff(float y, float m) {
  if (y == __int_as_float(0xff800000)) return 0.0f;
  const float t = __fsub_rn(y, m);
  const float bb = __fsub_rn(t, y);                                       // ~ -m
  const float err = __fadd_rn(__fsub_rn(y, __fsub_rn(t, bb)), __fsub_rn(-m, bb));  // (y - m) - t, exact
  const float e = expf(t);
  return __fmaf_rn(e, err, e);
}

// Fixed-point weight of the inverse-CDF sampler: floor(w * 2^40) for w >= 0, 0 otherwise.
__device__ __forceinline__ uint64_t fixed_weight(float w) {
  return w > 0.0f ? __float2ull_rz(__fmul_rn(w, 1099511627776.0f)) : 0ull;
}

// ------------------------------------------------------------------------------------------------
// Group-wide primitives.  A "group" is NT threads (a multiple of 32) of one CTA whose ranks 0..NT-1
// are passed in as `tid`; they synchronise on named barrier BAR so that other warps of the CTA
// (copy producers) are not involved.  `scratch` points to at least 2*(NT/32)+2 uint64 slots.
// ------------------------------------------------------------------------------------------------
template <int NT, int BAR>
__device__ __forceinline__ void group_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// OR of a predicate over the group (also a barrier).
template <int NT, int BAR>
__device__ __forceinline__ bool group_any(bool pred) {
  if (BAR == 0) return __syncthreads_or(pred ? 1 : 0) != 0;
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)(pred ? 1 : 0)), "n"(BAR), "n"(NT)
      : "memory");
  return r != 0;
}

__device__ __forceinline__ uint64_t shfl_u64(uint64_t v, int src) {
  const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)v, src);
  const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(v >> 32), src);
  return (uint64_t)lo | ((uint64_t)hi << 32);
}
__device__ __forceinline__ uint64_t shfl_up_u64(uint64_t v, int d) {
  const uint32_t lo = __shfl_up_sync(0xffffffffu, (uint32_t)v, d);
  const uint32_t hi = __shfl_up_sync(0xffffffffu, (uint32_t)(v >> 32), d);
  return (uint64_t)lo | ((uint64_t)hi << 32);
}

// Exclusive prefix sum of one value per thread in rank order; *total receives the group sum.
template <int NT, int BAR, typename T>
__device__ __forceinline__ T group_exclusive_scan(T v, int tid, uint64_t* scratch, T* total) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
  T inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    T n;
    if (sizeof(T) == 8) n = (T)shfl_up_u64((uint64_t)inc, d);
    else n = (T)__shfl_up_sync(0xffffffffu, (uint32_t)inc, d);
    if (lane >= d) inc += n;
  }
  if (lane == 31) scratch[warp] = (uint64_t)inc;
  group_sync<NT, BAR>();
  if (warp == 0) {
    uint64_t w = lane < NW ? scratch[lane] : 0;
    uint64_t winc = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint64_t n = shfl_up_u64(winc, d);
      if (lane >= d) winc += n;
    }
    if (lane < NW) scratch[NW + lane] = winc - w;
    if (lane == 31) scratch[2 * NW] = winc;
  }
  group_sync<NT, BAR>();
  const T warp_base = (T)scratch[NW + warp];
  *total = (T)scratch[2 * NW];
  const T result = warp_base + inc - v;
  group_sync<NT, BAR>();  // scratch may be reused immediately by the caller
  return result;
}

template <int NT, int BAR>
__device__ __forceinline__ uint64_t group_sum_u64(uint64_t v, int tid, uint64_t* scratch) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)v, d);
    const uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(v >> 32), d);
    v += (uint64_t)lo | ((uint64_t)hi << 32);
  }
  if (lane == 0) scratch[warp] = v;
  group_sync<NT, BAR>();
  uint64_t t = 0;
#pragma unroll
  for (int w = 0; w < NW; ++w) t += scratch[w];
  group_sync<NT, BAR>();
  return t;
}

template <int NT, int BAR>
__device__ __forceinline__ float group_sum_f32(float v, int tid, uint64_t* scratch) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
  float* f = reinterpret_cast<float*>(scratch);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  if (lane == 0) f[warp] = v;
  group_sync<NT, BAR>();
  // fixed-shape pairwise tree over the warp sums so that every thread gets the same value
  float w = lane < NW ? f[lane] : 0.0f;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) w += __shfl_xor_sync(0xffffffffu, w, d);
  group_sync<NT, BAR>();
  return w;
}

template <int NT, int BAR>
__device__ __forceinline__ float group_max_f32(float v, int tid, uint64_t* scratch) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
  float* f = reinterpret_cast<float*>(scratch);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
  if (lane == 0) f[warp] = v;
  group_sync<NT, BAR>();
  float w = lane < NW ? f[lane] : __int_as_float(0xff800000);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) w = fmaxf(w, __shfl_xor_sync(0xffffffffu, w, d));
  group_sync<NT, BAR>();
  return w;
}

// Fixed-point inverse-CDF draw over n entries in index order.  weight(k) returns the fixed-point
// weight of entry k (it is evaluated twice).  Returns the selected index to every thread, or -1 when
// the weights sum to zero.  scratch: 2*(NT/32)+4 uint64 slots.
template <int NT, int BAR, typename WeightFn>
__device__ __forceinline__ int group_icdf(WeightFn weight, int n, uint64_t R, int tid, uint64_t* scratch) {
  constexpr int ITEMS = 4;
  uint64_t local = 0;
  for (int k = tid; k < n; k += NT) local += weight(k);
  const uint64_t T = group_sum_u64<NT, BAR>(local, tid, scratch);
  if (T == 0) return -1;
  const uint64_t t = __umul64hi(R, T);
  int* found = reinterpret_cast<int*>(scratch + 2 * (NT / 32) + 2);
  uint64_t base = 0;
  for (int c0 = 0; c0 < n; c0 += NT * ITEMS) {
    const int k0 = c0 + tid * ITEMS;
    uint64_t w[ITEMS];
    uint64_t sum = 0;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      w[j] = (k0 + j < n) ? weight(k0 + j) : 0ull;
      sum += w[j];
    }
    uint64_t total;
    const uint64_t lo = base + group_exclusive_scan<NT, BAR, uint64_t>(sum, tid, scratch, &total);
    if (t >= lo && t < lo + sum) {
      uint64_t run = lo;
      int k = k0;
#pragma unroll
      for (int j = 0; j < ITEMS; ++j) {
        run += w[j];
        if (t < run) break;
        ++k;
      }
      *found = k;
    }
    base += total;
    if (t < base) break;  // uniform: every thread sees the same base
  }
  group_sync<NT, BAR>();
  const int k = *found;
  group_sync<NT, BAR>();
  return k;
}

// ------------------------------------------------------------------------------------------------
// One-barrier variants.  `scratch` holds two banks of 32 uint64 that successive calls alternate
// between (`flip`, kept by the caller, starts at 0 and must be passed to every call of the group in the
// same order by all its threads): a thread can be at most one barrier ahead of the slowest one, so
// the bank it writes is never the one a slower thread still reads.
// ------------------------------------------------------------------------------------------------
template <int NT, int BAR, typename T>
__device__ __forceinline__ T group_scan1(T v, int tid, uint64_t* scratch, int& flip, T* total) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
  T inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    T n;
    if (sizeof(T) == 8) n = (T)shfl_up_u64((uint64_t)inc, d);
    else n = (T)__shfl_up_sync(0xffffffffu, (uint32_t)inc, d);
    if (lane >= d) inc += n;
  }
  uint64_t* bank = scratch + (flip ? 32 : 0);
  flip ^= 1;
  if (lane == 31) bank[warp] = (uint64_t)inc;
  group_sync<NT, BAR>();
  // every warp scans the warps' totals for itself, lane w holding warp w's (a walk over the NW words by
  // every thread costs several times the instructions)
  const T x = lane < NW ? (T)bank[lane] : (T)0;
  T xi = x;
#pragma unroll
  for (int d = 1; d < NW; d <<= 1) {
    T n;
    if (sizeof(T) == 8) n = (T)shfl_up_u64((uint64_t)xi, d);
    else n = (T)__shfl_up_sync(0xffffffffu, (uint32_t)xi, d);
    if (lane >= d) xi += n;
  }
  T tot, base;
  if (sizeof(T) == 8) {
    tot = (T)shfl_u64((uint64_t)xi, NW - 1);
    base = (T)shfl_u64((uint64_t)(xi - x), warp);
  } else {
    tot = (T)__shfl_sync(0xffffffffu, (uint32_t)xi, NW - 1);
    base = (T)__shfl_sync(0xffffffffu, (uint32_t)(xi - x), warp);
  }
  *total = tot;
  return base + inc - v;
}

// Sum in a fixed order (lanes by butterfly, warps in index order): the same value in every thread and in
// every run.
template <int NT, int BAR>
__device__ __forceinline__ float group_sum1_f32(float v, int tid, uint64_t* scratch, int& flip) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  float* bank = reinterpret_cast<float*>(scratch + (flip ? 32 : 0));
  flip ^= 1;
  if (lane == 0) bank[warp] = v;
  group_sync<NT, BAR>();
  if ((NW & (NW - 1)) == 0) {
    // lane l takes warp (l mod NW)'s sum; the butterfly adds the same pairs in every lane and every warp
    float t = bank[lane & (NW - 1)];
#pragma unroll
    for (int d = NW / 2; d > 0; d >>= 1) t += __shfl_xor_sync(0xffffffffu, t, d);
    return t;
  }
  float t = 0.0f;
#pragma unroll
  for (int w = 0; w < NW; ++w) t += bank[w];
  return t;
}

template <int NT, int BAR>
__device__ __forceinline__ float group_max1_f32(float v, int tid, uint64_t* scratch, int& flip) {
  constexpr int NW = NT / 32;
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
  float* bank = reinterpret_cast<float*>(scratch + (flip ? 32 : 0));
  flip ^= 1;
  if (lane == 0) bank[warp] = v;
  group_sync<NT, BAR>();
  float t = __int_as_float(0xff800000);
#pragma unroll
  for (int w = 0; w < NW; ++w) t = fmaxf(t, bank[w]);
  return t;
}

}  // namespace sjd

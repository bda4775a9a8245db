// Row kernel with one contiguous range of token ids per filter thread.
//
// Same three roles per CTA as rows_pipeline_kernel (producer / filter / finisher, one persistent CTA per
// SM) and the same arithmetic; what differs is how a row is cut up.  The row of V logits is viewed as a
// matrix of 256 ranges x R ids (R = V/256): filter thread t owns ids [t R, (t+1) R).  A ring stage is a
// column slice of that matrix, 64 bytes per range, fetched by ONE tiled TMA copy per logits array
// (cp.async.bulk.tensor, box {64 bytes, 256 ranges, 1 row}, 64-byte swizzle so that the 16-byte reads of
// neighbouring threads fall into different banks).  Consequences:
//
//   * stage 0 of a row is a systematic sample of it (64 bytes out of every R elements), so the sampling
//     needs no schedule of its own;
//   * a thread meets its ids in ascending order and thread t's ids all precede thread t+1's: the hit bits
//     give the ids directly (id = t R + 2 * pair index) and the concatenation of the threads' lists IS the
//     ascending-id order.  The finisher therefore needs no bitmap, no prefix over it and no scatter: it
//     compacts the lists once, finds the exact K-th largest, and emits the survivors in list order.
//
// Shapes: V = 256 R with R a multiple of the stage width (32 bf16 / 16 fp32 elements) and 2..16 stages per
// row, rows at one uniform pitch.  Everything else goes to rows_pipeline_kernel or rows_generic_kernel.
#pragma once

#include <cuda.h>

#include "rows_pipeline.cuh"

namespace sjd {

constexpr int kRangeThreads = 256;          // filter threads = ranges per row
constexpr int kRangeStageBytes = 16384;     // one logits array in a ring stage: 64 bytes x 256 ranges
constexpr int kRangeRingStages = 3;
constexpr int kRangeDenseCap = 3584;        // candidates the finisher can hold for a row

struct RangeCfg {
  int sample_rank;  // m: rank (from the top) within the sample (stage 0) that fixes tau0
  int sample_all;   // 1: the first pass bins every sample element (m exceeds the number of groups of eight)
  int stages;       // S = R / (elements per stage and range)
  int range_len;    // R
  int mask_words;   // 32 hit bits each: R/2 pairs per range
};

enum {
  kRcAbort = 0,
  kRcFBin, kRcFAbove, kRcFCount, kRcSmaxKey,          // filter
  kRcRowTau0, kRcRowVmax, kRcRowTotal, kRcRowFallback,  // handed over with the row
  kRcPBin, kRcPAbove, kRcPCount, kRcGather, kRcPtok, kRcFoundId, kRcFoundP,  // finisher
  kRcWords = 20
};

struct BinMember {  // member of the threshold bin: value and where it sits in the dense list
  float y;
  int32_t slot;
};

struct RangeSmem {
  unsigned char* ring;  // [kRangeRingStages][2][kRangeStageBytes], 1024-byte aligned
  uint64_t* ylist;      // [kListCap][256] pair entries, one column per filter thread
  uint32_t* masks;      // [mask_words][256] inverted hit bits, first pair in the top bit
  Candidate* dense;     // [kRangeDenseCap] candidates in ascending id order
  int32_t* st_ids;      // [kKcapMax] survivors, ascending id
  float* st_vals;       // [kKcapMax]
  uint32_t* sel;        // [kSelBins]  = st_ids: dead before the survivors are staged
  BinMember* binlist;   // [kBinListCap] = st_vals: likewise
  uint32_t* hist;       // [kHistBins] filter
  uint64_t* full;       // [kRangeRingStages]
  uint64_t* empty;      // [kRangeRingStages]
  uint64_t* cand_full;
  uint64_t* cand_free;
  uint64_t* scan_f;
  uint64_t* scan_p;
  int* ctl;
};

__host__ __device__ inline size_t range_smem_bytes(int mask_words) {
  size_t b = 1024;  // alignment slack for the swizzled ring
  b += (size_t)kRangeRingStages * 2 * kRangeStageBytes;
  b += (size_t)kListCap * kRangeThreads * 8;
  b += (size_t)mask_words * kRangeThreads * 4;
  b += (size_t)kRangeDenseCap * sizeof(Candidate);
  b += (size_t)kKcapMax * 8;
  b += (size_t)kHistBins * 4;
  b += 16 * 8 + 2 * (2 * 32 + 8) * 8 + kRcWords * 4;
  return b;
}

__device__ __forceinline__ RangeSmem carve_range_smem(unsigned char* base, int mask_words) {
  static_assert(sizeof(uint32_t) * kSelBins <= sizeof(int32_t) * kKcapMax, "sel must fit under st_ids");
  static_assert(sizeof(BinMember) * kBinListCap <= sizeof(float) * kKcapMax, "binlist must fit under st_vals");
  RangeSmem s;
  unsigned char* p = base + ((1024u - (smem_u32(base) & 1023u)) & 1023u);
  s.ring = p;
  p += (size_t)kRangeRingStages * 2 * kRangeStageBytes;
  s.ylist = reinterpret_cast<uint64_t*>(p);
  p += (size_t)kListCap * kRangeThreads * 8;
  s.dense = reinterpret_cast<Candidate*>(p);
  p += (size_t)kRangeDenseCap * sizeof(Candidate);
  s.st_ids = reinterpret_cast<int32_t*>(p);
  s.sel = reinterpret_cast<uint32_t*>(p);
  p += (size_t)kKcapMax * 4;
  s.st_vals = reinterpret_cast<float*>(p);
  s.binlist = reinterpret_cast<BinMember*>(p);
  p += (size_t)kKcapMax * 4;
  s.hist = reinterpret_cast<uint32_t*>(p);
  p += (size_t)kHistBins * 4;
  s.masks = reinterpret_cast<uint32_t*>(p);
  p += (size_t)mask_words * kRangeThreads * 4;
  s.full = reinterpret_cast<uint64_t*>(p);
  s.empty = s.full + kRangeRingStages;
  s.cand_full = s.empty + kRangeRingStages;
  s.cand_free = s.cand_full + 1;
  p += 16 * 8;
  s.scan_f = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.scan_p = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.ctl = reinterpret_cast<int*>(p);
  return s;
}

// One tiled copy global -> shared: box {stage width, 256 ranges, 1 row} at element x of every range of
// row z.  x times the element size is a multiple of 64 bytes.  No multicast, own CTA only.
__device__ __forceinline__ void tma_load_box(void* dst, const CUtensorMap* map, int x, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(0), "r"(z), "r"(smem_u32(bar))
      : "memory");
}

// ---------------------------------------------------------------------------------------------------
// filter warps
// ---------------------------------------------------------------------------------------------------
template <int DTYPE, bool HAS_U, bool HAS_T>
__device__ __forceinline__ void range_filter_role(const RowArgs& a, const RangeCfg& cfg, const RangeSmem& sm, int tid) {
  constexpr int NT_F = kRangeThreads;
  constexpr int BAR_F = 1;
  constexpr uint32_t kStride = NT_F * 8;         // bytes between consecutive entries of one filter thread
  constexpr int TI = DTYPE != 0 ? 4 : 2;          // groups of eight elements per stage and thread
  constexpr int NS = kRangeRingStages;
  const int lane = tid & 31;
  const int mask_words = cfg.mask_words;
  const int rows = a.B * a.W;
  const float neg_inf = __int_as_float(0xff800000);
  const float lowest = -3.402823466e38f;  // with this threshold every finite value is a candidate
  volatile int* abort_flag = sm.ctl + kRcAbort;
  const uint64_t s2 = pack2(a.s, a.s), t2 = pack2(a.inv_T, a.inv_T);
  const uint32_t ring_addr = smem_u32(sm.ring);
  const uint32_t my_row = (uint32_t)tid * 64u;           // this thread's 64 bytes inside a staged array
  const uint32_t swz = ((uint32_t)tid >> 1) & 3u;        // 64-byte swizzle: 16-byte piece j sits at j ^ swz
  const uint32_t list_base = smem_u32(sm.ylist) + (uint32_t)tid * 8u;
  const uint32_t list_limit = list_base + (uint32_t)(kListCap - 4) * kStride;  // beyond it a group may not fit
  int slot = 0, flip = 0;
  uint32_t phase = 0;
  uint32_t n_row = 0;
  bool dead = false;

  // the j-th group of eight elements of this thread in the staged slice at `stage`
  auto load_group = [&](uint32_t stage, int j, RawTile<DTYPE>& r) {
    if (DTYPE != 0) {
      r.c[0] = lds128(stage + my_row + (((uint32_t)j ^ swz) << 4));
      if (HAS_U) r.u[0] = lds128(stage + kRangeStageBytes + my_row + (((uint32_t)j ^ swz) << 4));
    } else {
      r.c[0] = lds128(stage + my_row + (((uint32_t)(2 * j) ^ swz) << 4));
      r.c[DTYPE != 0 ? 0 : 1] = lds128(stage + my_row + (((uint32_t)(2 * j + 1) ^ swz) << 4));
      if (HAS_U) {
        r.u[0] = lds128(stage + kRangeStageBytes + my_row + (((uint32_t)(2 * j) ^ swz) << 4));
        r.u[DTYPE != 0 ? 0 : 1] = lds128(stage + kRangeStageBytes + my_row + (((uint32_t)(2 * j + 1) ^ swz) << 4));
      }
    }
  };

  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    // from the block's last row on, the verification grid may be scheduled (it waits for this grid's end)
    if (row + (int)gridDim.x >= rows) allow_dependent_launch();
    const int b = row / a.W, i = row - b * a.W;
    const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
    if (i >= L || dead) continue;

    // ---------------- stage 0 is the sample.  First pass: maxima of groups of eight, by key ----------------
    bool ok = mbar_wait(&sm.full[slot], phase);
    float smax = neg_inf;
    const uint32_t stage0 = ring_addr + (uint32_t)slot * (2 * kRangeStageBytes);
    if (ok) {
#pragma unroll
      for (int j = 0; j < TI; ++j) {
        RawTile<DTYPE> raw;
        load_group(stage0, j, raw);
        float y[8];
        merge_raw<DTYPE, HAS_U, HAS_T>(raw, s2, t2, y);
        const float m8 = max3(max3(max3(neg_inf, y[0], y[1]), y[2], y[3]), max3(y[4], y[5], y[6]), y[7]);
        if (cfg.sample_all) {
#pragma unroll
          for (int k = 0; k < 8; ++k) atomicAdd(&sm.hist[float_key(canonical(y[k])) >> 21], 1u);
        } else {
          atomicAdd(&sm.hist[float_key(canonical(m8)) >> 21], 1u);
        }
        smax = fmaxf(smax, m8);
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, d));
    if (lane == 0) atomicMax(reinterpret_cast<unsigned int*>(&sm.ctl[kRcSmaxKey]), float_key(canonical(smax)));
    dead = group_any<NT_F, BAR_F>(!ok);
    if (dead) {
      if (tid == 0) *abort_flag = 1;
      continue;
    }
    // at least m group maxima (or, binning everything, m elements), hence at least m sample elements, are >=
    // the lower edge of this bin
    find_rank_bin<kHistBins, NT_F, BAR_F>(sm.hist, (uint32_t)cfg.sample_rank, tid, sm.scan_f, flip, sm.ctl, kRcFBin);
    const int cbin = sm.ctl[kRcFBin];
    float floor_y = cbin >= 0 ? key_float((uint32_t)cbin << 21) : lowest;
    if (!(floor_y >= lowest)) floor_y = lowest;  // edge fell on -inf or into the NaN patterns
    const float top_y = key_float((uint32_t)sm.ctl[kRcSmaxKey]);
    const bool refine = floor_y > lowest && top_y >= floor_y && top_y <= 3.402823466e38f;
    const float range = __fsub_rn(top_y, floor_y);
    const float scale = (refine && range > 0.0f) ? __fdiv_rn((float)kHistBins - 0.5f, range) : 0.0f;

    uint32_t cur = list_base;  // shared-memory address of the thread's next free entry
    uint32_t imw = 0;          // inverted hit bits of the groups filtered since the last full mask word
    bool overflow = false;
    // One group: four pairs.  A pair is always stored at the cursor; the cursor moves on only for a hit,
    // i.e. when max(pair) >= thr.  A pair of NaNs and -inf never hit.
    auto filter_group = [&](const RawTile<DTYPE>& raw, float thr) {
      float y[8];
      merge_raw<DTYPE, HAS_U, HAS_T>(raw, s2, t2, y);
      if (cur > list_limit) {
        overflow = true;
        cur = list_base;
      }
      uint32_t d = cur;
      imw <<= 4;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float m = fmaxf(y[2 * k], y[2 * k + 1]);
        asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(d), "f"(y[2 * k]), "f"(y[2 * k + 1]) : "memory");
        // hit: the cursor moves on; miss: the pair's bit is set in the inverted mask (both predicated, no branch)
        asm("{\n\t.reg .pred p;\n\tsetp.ge.f32 p, %2, %3;\n\t@p add.u32 %0, %0, %4;\n\t@!p or.b32 %1, %1, %5;\n\t}"
            : "+r"(d), "+r"(imw)
            : "f"(m), "f"(thr), "r"(kStride), "r"(8u >> k));
      }
      cur = d;
    };
    // after stage s the thread has filtered (s + 1) TI groups; every eight groups fill one mask word
    auto end_stage = [&](int s) {
      const int done = (s + 1) * TI;
      if ((done & 7) == 0) {
        if ((done >> 3) <= mask_words) sm.masks[(size_t)((done >> 3) - 1) * NT_F + tid] = imw;
        imw = 0;
      }
    };
    // ---------------- the sample against the floor (a superset of what tau0 will keep) ----------------
    const float sample_thr = refine ? floor_y : lowest;
#pragma unroll
    for (int j = 0; j < TI; ++j) {
      RawTile<DTYPE> raw;
      load_group(stage0, j, raw);
      filter_group(raw, sample_thr);
    }
    end_stage(0);
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[slot]);
    if (++slot == NS) {
      slot = 0;
      phase ^= 1u;
    }
    // ---------------- second pass: linear bins over [floor, sample max], from the lists ----------------
    float tau0 = lowest;
    if (refine) {
      for (uint32_t e = list_base; e < cur; e += kStride) {
        float v0, v1;
        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v0), "=f"(v1) : "r"(e));
        if (v0 >= floor_y) {
          const int q = __float2int_rd(__fmul_rn(__fsub_rn(v0, floor_y), scale));
          atomicAdd(&sm.hist[min(max(q, 0), kHistBins - 1)], 1u);
        }
        if (v1 >= floor_y) {
          const int q = __float2int_rd(__fmul_rn(__fsub_rn(v1, floor_y), scale));
          atomicAdd(&sm.hist[min(max(q, 0), kHistBins - 1)], 1u);
        }
      }
      group_sync<NT_F, BAR_F>();
      if (tid == 0) sm.ctl[kRcSmaxKey] = 0;  // every thread has read it; next written after the next row's barriers
      find_rank_bin<kHistBins, NT_F, BAR_F>(sm.hist, (uint32_t)cfg.sample_rank, tid, sm.scan_f, flip, sm.ctl, kRcFBin);
      const int fbin = sm.ctl[kRcFBin];
      if (fbin > 0 && scale > 0.0f) {
        // a little below the lower edge of the bin, so that rounding cannot exclude one of its members
        const float t = __fmul_rd(__fdiv_rd((float)fbin, scale), 0.99999f);
        tau0 = __fadd_rd(floor_y, t);
      } else if (fbin >= 0) {
        tau0 = floor_y;
      }
    } else {
      group_sync<NT_F, BAR_F>();
      if (tid == 0) sm.ctl[kRcSmaxKey] = 0;
    }
    // ---------------- the rest of the row against tau0 ----------------
    for (int s = 1; s < cfg.stages; ++s) {
      if (ok) ok = mbar_wait(&sm.full[slot], phase);
      if (ok) {
        const uint32_t stage = ring_addr + (uint32_t)slot * (2 * kRangeStageBytes);
        RawTile<DTYPE> raw[TI];
#pragma unroll
        for (int j = 0; j < TI; ++j) load_group(stage, j, raw[j]);
#pragma unroll
        for (int j = 0; j < TI; ++j) filter_group(raw[j], tau0);
        end_stage(s);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[slot]);
      if (++slot == NS) {
        slot = 0;
        phase ^= 1u;
      }
    }
    // ---------------- drain: this thread's list becomes its run of the dense list ----------------
    // Threads own ascending id ranges and meet their ids in ascending order, so writing the runs one
    // after the other yields the candidates in ascending id order.
    {
      const int it = cfg.stages * TI;  // groups of eight this thread has filtered in this row
      const int rem = it & 7;
      int w = it >> 3;
      if (rem != 0 && w < mask_words) {
        const int fill = 32 - 4 * rem;  // bits of the word not reached: misses
        sm.masks[(size_t)w * NT_F + tid] = (imw << fill) | ((1u << fill) - 1u);
        ++w;
      }
      for (; w < mask_words; ++w) sm.masks[(size_t)w * NT_F + tid] = 0xffffffffu;
    }
    const int n_e = overflow ? 0 : (int)((cur - list_base) / kStride);
    uint32_t my_valid = 0;
    float vmax = neg_inf;
    for (int e = 0; e < n_e; ++e) {
      float v0, v1;
      asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v0), "=f"(v1) : "r"(list_base + (uint32_t)e * kStride));
      if (v0 >= tau0) {
        ++my_valid;
        vmax = fmaxf(vmax, v0);
      }
      if (v1 >= tau0) {
        ++my_valid;
        vmax = fmaxf(vmax, v1);
      }
    }
    uint32_t n_total;
    uint32_t my_off = group_scan1<NT_F, BAR_F, uint32_t>(my_valid, tid, sm.scan_f, flip, &n_total);
    vmax = group_max1_f32<NT_F, BAR_F>(vmax, tid, sm.scan_f, flip);
    // the dense list must be back from the finisher
    if (ok && n_row > 0) ok = mbar_wait(sm.cand_free, (n_row - 1) & 1u);
    const bool any_overflow = group_any<NT_F, BAR_F>(overflow);
    dead = group_any<NT_F, BAR_F>(!ok);
    if (dead) {
      if (tid == 0) *abort_flag = 1;
      continue;  // the row is not handed over: the finisher's wait runs out and marks the rows
    }
    // too few candidates (the sampled threshold was too high), too many for the list, or no finite maximum:
    // the finisher redoes the row by the any-shape path
    const bool fallback = any_overflow || n_total < (uint32_t)a.kcap || n_total > (uint32_t)kRangeDenseCap ||
                          !(vmax <= 3.402823466e38f);
    if (!fallback) {
      const int id0 = tid * cfg.range_len;
      int e = 0;
      for (int w = 0; w < mask_words; ++w) {
        uint32_t x = ~sm.masks[(size_t)w * NT_F + tid];
        while (x != 0u && e < n_e) {
          const int bitpos = __clz((int)x);
          x &= ~(0x80000000u >> bitpos);
          const int id = id0 + 2 * (w * 32 + bitpos);  // pair q of range t holds ids t R + 2q and t R + 2q + 1
          float v0, v1;
          asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v0), "=f"(v1) : "r"(list_base + (uint32_t)e * kStride));
          ++e;
          if (v0 >= tau0) sm.dense[my_off++] = Candidate{canonical(v0), id};
          if (v1 >= tau0) sm.dense[my_off++] = Candidate{canonical(v1), id + 1};
        }
      }
    }
    group_sync<NT_F, BAR_F>();
    if (tid == 0) {
      sm.ctl[kRcRowTau0] = __float_as_int(tau0);
      sm.ctl[kRcRowVmax] = __float_as_int(vmax);
      sm.ctl[kRcRowTotal] = (int)n_total;
      sm.ctl[kRcRowFallback] = fallback ? 1 : 0;
      mbar_arrive(sm.cand_full);
    }
    ++n_row;
  }
}

// ---------------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------------
template <int DTYPE, int NP>
__global__ void __launch_bounds__((8 + NP + 1) * 32, 1)
rows_ranges_kernel(const RowArgs a, const RangeCfg cfg, const __grid_constant__ CUtensorMap map_c,
                   const __grid_constant__ CUtensorMap map_u) {
  constexpr int NF = 8;
  constexpr int NT_F = kRangeThreads, NT_P = NP * 32;
  constexpr int BAR_P = 2;  // named barrier of the finisher warps (the filter warps use 1)
  constexpr int kFinItems = kKcapMax / NT_P;
  constexpr int NS = kRangeRingStages;
  constexpr int BW = 64 / (DTYPE != 0 ? 2 : 4);  // elements per stage and range
  static_assert(NT_F == NF * 32 && kFinItems == 8, "group sizes");
  extern __shared__ unsigned char smem_raw[];
  RangeSmem sm = carve_range_smem(smem_raw, cfg.mask_words);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool has_u = a.uncond != nullptr;
  const float neg_inf = __int_as_float(0xff800000);
  const int rows = a.B * a.W;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], NF);
    }
    mbar_init(sm.cand_full, 1);
    mbar_init(sm.cand_free, 1);
    for (int k = 0; k < kRcWords; ++k) sm.ctl[k] = 0;
    fence_barrier_init();
  }
  for (int j = threadIdx.x; j < kHistBins; j += blockDim.x) sm.hist[j] = 0;
  for (int j = threadIdx.x; j < kSelBins; j += blockDim.x) sm.sel[j] = 0;
  // everything above touched shared memory only; global memory is read and written from here on, so a
  // launch that was allowed to overlap the previous kernel of the stream waits for that kernel's end here
  grid_dependency_wait();
  __syncthreads();
  volatile int* abort_flag = sm.ctl + kRcAbort;

  if (warp == NF + NP) {
    // ====================================== producer warp ======================================
    if (lane != 0) return;
    int slot = 0;
    uint32_t use = 0, issued = 0;
    bool ok = true;
    const uint32_t stage_bytes = (uint32_t)kRangeStageBytes * (has_u ? 2u : 1u);
    for (int row = blockIdx.x; row < rows && ok; row += gridDim.x) {
      const int b = row / a.W, i = row - b * a.W;
      const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
      if (i >= L) continue;
      for (int s = 0; s < cfg.stages; ++s) {
        if (use > 0) ok = mbar_wait(&sm.empty[slot], (use - 1) & 1u);
        ok = ok && (*abort_flag == 0);
        if (!ok) break;
        unsigned char* dst = sm.ring + (size_t)slot * (2 * kRangeStageBytes);
        mbar_arrive_expect_tx(&sm.full[slot], stage_bytes);
        tma_load_box(dst, &map_c, s * BW, row, &sm.full[slot]);
        if (has_u) tma_load_box(dst + kRangeStageBytes, &map_u, s * BW, row, &sm.full[slot]);
        ++issued;
        if (++slot == NS) {
          slot = 0;
          ++use;
        }
      }
    }
    // drain: every stage armed here must have landed before the CTA may exit
    {
      const uint32_t n_back = issued < (uint32_t)NS ? issued : (uint32_t)NS;
      int sl = slot;
      uint32_t us = use;
      for (uint32_t k = 0; k < n_back; ++k) {
        if (--sl < 0) {
          sl = NS - 1;
          --us;
        }
        mbar_wait(&sm.full[sl], us & 1u);
      }
      if (!ok) *abort_flag = 1;
    }
    return;
  }

  if (warp < NF) {
    // ======================================= filter warps =======================================
    const bool has_t = a.inv_T != 1.0f;
    if (has_u) {
      if (has_t) range_filter_role<DTYPE, true, true>(a, cfg, sm, threadIdx.x);
      else range_filter_role<DTYPE, true, false>(a, cfg, sm, threadIdx.x);
    } else {
      if (has_t) range_filter_role<DTYPE, false, true>(a, cfg, sm, threadIdx.x);
      else range_filter_role<DTYPE, false, false>(a, cfg, sm, threadIdx.x);
    }
    return;
  }

  // ======================================= finisher warps =======================================
  const int tid = threadIdx.x - NT_F;  // 0 .. NT_P-1; also the filter thread whose list this thread drains
  int flip = 0;
  uint32_t n_row = 0;
  bool dead = false;
  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    // from the block's last row on, the verification grid may be scheduled (it waits for this grid's end)
    if (row + (int)gridDim.x >= rows) allow_dependent_launch();
    const int b = row / a.W, i = row - b * a.W;
    const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
    RowScratch* rs = a.scratch + row;
    if (i >= L) {
      if (tid == 0) {
        a.out_cnt[row] = 0;
        *rs = RowScratch{0.0f, -1, 0.0f, 0};
      }
      continue;
    }
    const int kcap = a.kcap;
    const int draft = a.drafts ? a.drafts[row] : -1;
    // the row's own random number: needed last, computed while waiting
    const int pos = (a.pos_base ? a.pos_base[b] : 0) + i;
    const int iter = a.iteration ? a.iteration[b] : a.iteration0;
    const Philox4 rnd = philox4x32_10((uint32_t)pos, (uint32_t)(a.seq_base + b), (uint32_t)iter, (uint32_t)a.purpose,
                                      a.seed_lo, a.seed_hi);
    if (!dead) dead = !mbar_wait(sm.cand_full, n_row & 1u);
    dead = group_any<NT_P, BAR_P>(dead || (*abort_flag != 0));
    if (dead) {
      if (tid == 0) {
        *abort_flag = 1;
        a.out_cnt[row] = 0;
        *rs = RowScratch{0.0f, -1, 0.0f, kRowStatusTimeout};
      }
      continue;
    }
    const float tau0 = __int_as_float(sm.ctl[kRcRowTau0]);
    const float vmax = __int_as_float(sm.ctl[kRcRowVmax]);
    const uint32_t n_total = (uint32_t)sm.ctl[kRcRowTotal];
    bool fallback = kcap > kKcapMax || sm.ctl[kRcRowFallback] != 0;
    ++n_row;
    if (fallback) {
      // exact any-shape path from global memory (the row is still in L2); its scratch sits on st_vals, so
      // that the bins (= st_ids) stay clear
      group_sync<NT_P, BAR_P>();
      if (tid == 0) mbar_arrive(sm.cand_free);
      row_generic<DTYPE, NT_P, BAR_P>(a, row, tid, *reinterpret_cast<GenericSmem*>(sm.st_vals), kRowStatusRedone);
      continue;
    }
    // linear bins over [tau0, vmax]; monotone in y, so a higher bin never holds a smaller value
    const float range = __fsub_rn(vmax, tau0);
    const float scale = range > 0.0f ? __fdiv_rn((float)kSelBins * 0.999f, range) : 0.0f;
    auto bin_of = [&](float y) {
      const int q = __float2int_rd(__fmul_rn(__fsub_rn(y, tau0), scale));
      return min(max(q, 0), kSelBins - 1);
    };
    if (tid == 0) {
      sm.ctl[kRcGather] = 0;
      sm.ctl[kRcPtok] = 0;
      sm.ctl[kRcFoundId] = -1;
    }
    // every candidate into its bin, four independent entries per thread in flight
    for (uint32_t i0 = 0; i0 < n_total; i0 += 4 * NT_P) {
      float yv[4];
      bool v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint32_t ix = i0 + q * NT_P + tid;
        v[q] = ix < n_total;
        if (v[q]) yv[q] = sm.dense[ix].y;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (v[q]) atomicAdd(&sm.sel[bin_of(yv[q])], 1u);
    }
    group_sync<NT_P, BAR_P>();
    // ---- exact K-th largest: threshold bin, then ranking inside it by (y descending, id ascending) ----
    int tbin = 0, need = 0, nbin = 0;
    find_rank_bin<kSelBins, NT_P, BAR_P>(sm.sel, (uint32_t)kcap, tid, sm.scan_p, flip, sm.ctl, kRcPBin);
    if (!fallback) {
      tbin = sm.ctl[kRcPBin];
      need = kcap - sm.ctl[kRcPAbove];  // members of the threshold bin that survive
      nbin = sm.ctl[kRcPCount];
      if (tbin < 0 || nbin > kBinListCap) fallback = true;
    }
    // from here on every thread works on an equal share of the dense list: a run of consecutive entries,
    // so that concatenating the threads' survivors keeps the id order
    const uint32_t chunk = (n_total + NT_P - 1) / NT_P;
    const uint32_t my_first = fallback ? 0u : min((uint32_t)tid * chunk, n_total);
    const uint32_t my_count = fallback ? 0u : min(my_first + chunk, n_total) - my_first;
    uint32_t n_above = 0, n_in_bin = 0;
    if (!fallback) {
      for (uint32_t k = 0; k < my_count; ++k) {
        const Candidate c = sm.dense[my_first + k];
        const int q = bin_of(c.y);
        if (q > tbin) ++n_above;
        else if (q == tbin) {
          ++n_in_bin;
          sm.binlist[atomicAdd(&sm.ctl[kRcGather], 1)] = BinMember{c.y, (int32_t)(my_first + k)};
        }
      }
    }
    group_sync<NT_P, BAR_P>();
    if (!fallback) {
      // losers of the threshold bin are struck from the dense list: the sign bit of their id is set
      for (int x = tid; x < nbin; x += NT_P) {
        const BinMember me = sm.binlist[x];
        const int my_id = sm.dense[me.slot].id & 0x7fffffff;
        int rank = 0;
        for (int z = 0; z < nbin; ++z) {
          const BinMember o = sm.binlist[z];
          const int o_id = sm.dense[o.slot].id & 0x7fffffff;
          rank += (o.y > me.y || (o.y == me.y && o_id < my_id)) ? 1 : 0;
        }
        if (rank >= need) sm.dense[me.slot].id = my_id | (int)0x80000000;
      }
    }
    group_sync<NT_P, BAR_P>();
    uint32_t my_alive = n_above;
    if (n_in_bin != 0u) {
      for (uint32_t k = 0; k < my_count; ++k) {
        const Candidate c = sm.dense[my_first + k];
        if (c.id >= 0 && bin_of(c.y) == tbin) ++my_alive;
      }
    }
    uint32_t total_alive;
    uint32_t out_pos = group_scan1<NT_P, BAR_P, uint32_t>(my_alive, tid, sm.scan_p, flip, &total_alive);
    if (!fallback && total_alive != (uint32_t)kcap) fallback = true;  // cannot happen; keep the result exact anyway
    if (!fallback) {
      // ---- survivors, already in ascending id order (this overwrites sel and binlist) ----
      for (uint32_t k = 0; k < my_count; ++k) {
        const Candidate c = sm.dense[my_first + k];
        if (c.id >= 0 && bin_of(c.y) >= tbin) {
          sm.st_ids[out_pos] = c.id;
          sm.st_vals[out_pos] = c.y;
          ++out_pos;
        }
      }
    }
    group_sync<NT_P, BAR_P>();
    // the dense list is not read again: hand it back
    if (tid == 0) mbar_arrive(sm.cand_free);
    if (fallback) {
      // the threshold bin was too crowded for the on-chip ranking: exact any-shape path from global memory.
      // The bins were cleared when they were read; the any-shape path's scratch sits on st_vals.
      for (int j = tid; j < kSelBins; j += NT_P) sm.sel[j] = 0;
      row_generic<DTYPE, NT_P, BAR_P>(a, row, tid, *reinterpret_cast<GenericSmem*>(sm.st_vals), kRowStatusRedone);
      continue;
    }
    // ---- normalise, write the row, draw from it ----
    const int k0 = tid * kFinItems;
    float e[kFinItems];
    int ids[kFinItems];
    float zpart = 0.0f;
#pragma unroll
    for (int j = 0; j < kFinItems; ++j) {
      const bool in = k0 + j < kcap;
      e[j] = in ? exp_diff(sm.st_vals[k0 + j], vmax) : 0.0f;
      ids[j] = in ? sm.st_ids[k0 + j] : -1;
      zpart += e[j];
    }
    // these words of st_ids are this thread's share of sel: zero again for the next row
    *reinterpret_cast<uint4*>(sm.sel + k0) = make_uint4(0u, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(sm.sel + k0 + 4) = make_uint4(0u, 0u, 0u, 0u);
    const float Z = group_sum1_f32<NT_P, BAR_P>(zpart, tid, sm.scan_p, flip);
    int32_t* out_ids = a.out_ids + (size_t)row * kcap;
    float* out_vals = a.out_vals + (size_t)row * kcap;
    uint64_t wgt[kFinItems], wloc = 0;
    float p[kFinItems];
#pragma unroll
    for (int j = 0; j < kFinItems; ++j) {
      p[j] = __fdiv_rn(e[j], Z);
      wgt[j] = fixed_weight(p[j]);
      wloc += wgt[j];
      if (ids[j] == draft && ids[j] >= 0) sm.ctl[kRcPtok] = __float_as_int(p[j]);
    }
    if ((kcap & 3) == 0 && k0 + kFinItems <= kcap) {
      int4* oi = reinterpret_cast<int4*>(out_ids + k0);
      float4* ov = reinterpret_cast<float4*>(out_vals + k0);
      oi[0] = make_int4(ids[0], ids[1], ids[2], ids[3]);
      oi[1] = make_int4(ids[4], ids[5], ids[6], ids[7]);
      ov[0] = make_float4(p[0], p[1], p[2], p[3]);
      ov[1] = make_float4(p[4], p[5], p[6], p[7]);
    } else {
#pragma unroll
      for (int j = 0; j < kFinItems; ++j) {
        if (k0 + j < kcap) {
          out_ids[k0 + j] = ids[j];
          out_vals[k0 + j] = p[j];
        }
      }
    }
    // the row's own draw from p_i: fixed-point inverse CDF in ascending-id order
    uint64_t T;
    const uint64_t lo = group_scan1<NT_P, BAR_P, uint64_t>(wloc, tid, sm.scan_p, flip, &T);
    const uint64_t t = __umul64hi(random64(rnd), T);
    if (T > 0 && t >= lo && t < lo + wloc) {
      uint64_t run = lo;
      int j = 0;
#pragma unroll
      for (int q = 0; q < kFinItems; ++q) {
        run += wgt[q];
        if (t >= run) j = q + 1;
      }
      // j < kFinItems because t < lo + wloc
      int fid = ids[0];
      float fp = p[0];
#pragma unroll
      for (int q = 1; q < kFinItems; ++q) {
        if (q == j) {
          fid = ids[q];
          fp = p[q];
        }
      }
      sm.ctl[kRcFoundId] = fid;
      sm.ctl[kRcFoundP] = __float_as_int(fp);
    }
    if (T == 0 && tid == 0) {  // all weights rounded to zero: take the first entry
      sm.ctl[kRcFoundId] = ids[0];
      sm.ctl[kRcFoundP] = __float_as_int(p[0]);
    }
    group_sync<NT_P, BAR_P>();
    if (tid == 0) {
      a.out_cnt[row] = kcap;
      *rs = RowScratch{__int_as_float(sm.ctl[kRcPtok]), sm.ctl[kRcFoundId], __int_as_float(sm.ctl[kRcFoundP]), 0};
    }
    group_sync<NT_P, BAR_P>();
  }
}

}  // namespace sjd

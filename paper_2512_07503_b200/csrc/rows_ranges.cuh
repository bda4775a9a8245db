// Row kernel with one contiguous range of token ids per filter thread.
//
// One persistent CTA per SM, rows round-robin, four roles:
//
//   producer (1 warp)   streams rows through a ring of shared-memory stages with tiled TMA copies.
//   sampler (3 warps)   works one row AHEAD of the filter: it gets a copy of the next row's stage 0 (a
//                       systematic sample of that row) through the ring, and turns it into the candidate
//                       threshold tau0 of that row while the filter warps are still streaming the current one.
//   filter (8 warps)    merges the staged pairs into logits y and keeps the pairs that reach tau0; at the end
//                       of the row it compacts its lists into a dense candidate list in ascending id order.
//   finisher (16 warps) one row BEHIND the filter: exact K-th largest among the candidates, softmax, output,
//                       the row's own draw.  Before the CTA's first row they compute that row's threshold.
//
// Every combination of (guidance given, temperature applied, thresholds by group maxima or by elements) is a
// kernel of its own, chosen on the host: the roles' code is large against the SM's instruction caches, and
// the variants a launch does not run cost time merely by lying between those it does.
//
// The row of V logits is viewed as a matrix of 256 ranges x R ids (R = V/256): filter thread t owns ids
// [t R, (t+1) R).  A ring stage is a column slice of that matrix, 64 bytes per range, fetched by ONE tiled
// TMA copy per logits array (cp.async.bulk.tensor, box {64 bytes, 256 ranges, 1 row}, 64-byte swizzle so
// that the 16-byte reads of neighbouring threads fall into different banks).  Consequences:
//
//   * stage 0 of a row is a systematic sample of it (64 bytes out of every R elements).  It is fetched
//     twice: once a row early for the sampler, once in its turn for the filter (by then it sits in L2).
//     Plain loads would not do for the sampler: behind the ring's outstanding copies they take thousands
//     of cycles each;
//   * a thread meets its ids in ascending order and thread t's ids all precede thread t+1's: the hit bits
//     give the ids directly (id = t R + 2 * pair index) and the concatenation of the threads' lists IS the
//     ascending-id order.  The finisher therefore needs no bitmap, no prefix over it and no scatter.
//
// Shapes: V = 256 R with R a multiple of the stage width (32 bf16 / 16 fp32 elements) and 2..16 stages per
// row, rows at one uniform pitch.  Everything else goes to rows_pipeline_kernel or rows_generic_kernel.
#pragma once

#include <cuda.h>

#include "rows_pipeline.cuh"

namespace sjd {

// Phase timers: with -DSJD_PHASE_TIMERS thread 0 of every role adds the clock cycles between two marks to a
// device-side table (read by sjd_phase_cycles_read); without it the marks compile to nothing.
#ifdef SJD_PHASE_TIMERS
__device__ unsigned long long g_phase_cycles[48];
#define SJD_PHASE_BEGIN() long long phase_t0_ = clock64()
#define SJD_PHASE(i)                                                                   \
  do {                                                                                 \
    if (tid == 0) {                                                                    \
      const long long phase_t_ = clock64();                                            \
      atomicAdd(&g_phase_cycles[i], (unsigned long long)(phase_t_ - phase_t0_));       \
      phase_t0_ = phase_t_;                                                            \
    }                                                                                  \
  } while (0)
#define SJD_PHASE_COUNT(i, n) \
  do {                        \
    if (tid == 0) atomicAdd(&g_phase_cycles[i], (unsigned long long)(n)); \
  } while (0)
#else
#define SJD_PHASE_BEGIN()
#define SJD_PHASE(i)
#define SJD_PHASE_COUNT(i, n)
#endif

constexpr int kRangeThreads = 256;          // filter threads = ranges per row
constexpr int kRangeStageBytes = 16384;     // one logits array in a ring stage: 64 bytes x 256 ranges
constexpr int kRangeRingStages = 3;
constexpr int kRangeListCap = 35;           // pair entries per filter thread and row (the last four are slack for
                                            // the unconditional stores of one group)
constexpr int kRangePairCap = 3328;         // candidate pairs the finisher can hold for a row
constexpr int kSampleBins = 1024;           // sampler's histogram (group maxima by key, then linear bins)
constexpr int kSampleKeyShift = 22;         // key bits dropped by the first histogram: sign, exponent, one mantissa bit
constexpr int kRowsPerCta = 32;             // live rows a CTA takes in one launch (the host splits larger problems)

struct RangeCfg {
  int sample_rank;  // m: rank (from the top) within the sample (stage 0) that fixes tau0
  int sample_all;   // 1: the first pass bins every sample element (m exceeds the number of groups of eight)
  int group_rank;   // > 0: tau0 is the group maximum of this rank (the element rank m translated, see the sampler)
  int stages;       // S = R / (elements per stage and range)
  int range_len;    // R
  int mask_words;   // 32 hit bits each: R/2 pairs per range
  int row_begin;    // this launch covers rows [row_begin, row_end)
  int row_end;
};

enum {
  kRcAbort = 0,
  kRcLive,                                              // live rows of this CTA (entries of the row table)
  kRcABin, kRcAAbove, kRcACount, kRcSmaxKey,           // sampler
  kRcBBin, kRcBSmaxKey,                                 // the first row's sampling, done by the finisher warps
  kRcTau0, kRcTau1, kRcTau2, kRcTau3,                   // tau0 of live row k in word kRcTau0 + (k & 3)
  kRcTop0, kRcTop1, kRcTop2, kRcTop3,                   // largest sample value of live row k, likewise
  kRcRowTau0, kRcRowTop, kRcRowPairs, kRcRowFallback,   // handed over with the row
  kRcPBin, kRcPAbove, kRcPCount, kRcGather, kRcPtok, kRcFoundId, kRcFoundP, kRcRedo, kRcRndLo, kRcRndHi,  // finisher
  kRcTrashA, kRcTrashB,                                 // where the histogram updates of lanes with nothing to count go
  kRcWords = 32
};

struct BinMember {  // member of the threshold bin: value and where it sits in the pair list (2 * pair + half)
  float y;
  int32_t slot;
};

struct RowEntry {  // one live row of this CTA with what the roles need to know about it
  int32_t row;    // b * W + i
  int32_t pos;    // absolute position of the row: pos_base[b] + i
  int32_t iter;   // iteration counter of its sequence
  int32_t draft;  // its draft token, -1 when every row is drafted
};

struct RangeSmem {
  unsigned char* ring;  // [kRangeRingStages][2][kRangeStageBytes], 1024-byte aligned
  uint64_t* ylist;      // [kRangeListCap][256] pair entries, one column per filter thread
  uint32_t* masks;      // [mask_words][256] inverted hit bits, first pair in the top bit
  uint64_t* pair_y;     // [kRangePairCap] candidate pairs {y(2q), y(2q+1)} in ascending id order
  uint16_t* pair_q;     // [kRangePairCap] their pair numbers q (ids 2q and 2q+1)
  int32_t* st_ids;      // [kKcapMax] survivors, ascending id
  float* st_vals;       // [kKcapMax]
  uint32_t* sel;        // [kSelBins]  = st_ids: dead before the survivors are staged
  BinMember* binlist;   // [kBinListCap] = st_vals: likewise
  uint32_t* hist;       // [kSampleBins] sampler
  uint32_t* hist_c;     // [kSampleBins / 32] its coarse level
  uint32_t* sel_c;      // [kSelBins / 32] coarse level of sel (and of the first row's sampling, which borrows sel)
  RowEntry* tab;        // [kRowsPerCta]
  int32_t* redo;        // [kRowsPerCta] rows the single pass could not finish (redone at the end)
  uint64_t* full;       // [kRangeRingStages] a row stage has landed in the slot (waited for by the filter)
  uint64_t* empty;      // [kRangeRingStages] the slot's eight consumer warps are done with it
  uint64_t* sample_full;  // [2] a sample has landed in its slot (row parity; waited for by the sampler)
  uint64_t* tau_full;   // [2] tau0 of a row published by the sampler (row parity)
  uint64_t* cand_full;
  uint64_t* cand_free;
  uint64_t* scan_f;
  uint64_t* scan_p;
  uint64_t* scan_a;
  int* ctl;
};

__host__ __device__ inline size_t range_smem_bytes(int mask_words) {
  size_t b = 1024;  // alignment slack for the swizzled ring
  b += (size_t)kRangeRingStages * 2 * kRangeStageBytes;
  b += (size_t)kRangeListCap * kRangeThreads * 8;
  b += (size_t)mask_words * kRangeThreads * 4;
  b += (size_t)kRangePairCap * (8 + 2);
  b += (size_t)kKcapMax * 8;
  b += (size_t)kSampleBins * 4;
  b += (size_t)kRowsPerCta * sizeof(RowEntry);
  b += (size_t)kRowsPerCta * 4;
  b += 16 * 8 + 3 * (2 * 32 + 8) * 8 + kRcWords * 4;
  b += (size_t)(kSampleBins / 32 + kSelBins / 32) * 4;
  return b;
}

__device__ __forceinline__ RangeSmem carve_range_smem(unsigned char* base, int mask_words) {
  static_assert(sizeof(uint32_t) * kSelBins <= sizeof(int32_t) * kKcapMax, "sel must fit under st_ids");
  static_assert(sizeof(BinMember) * kBinListCap <= sizeof(float) * kKcapMax, "binlist must fit under st_vals");
  static_assert((kRangePairCap * 2) % 16 == 0, "what follows the pair numbers stays 16-byte aligned");
  RangeSmem s;
  unsigned char* p = base + ((1024u - (smem_u32(base) & 1023u)) & 1023u);
  s.ring = p;
  p += (size_t)kRangeRingStages * 2 * kRangeStageBytes;
  s.ylist = reinterpret_cast<uint64_t*>(p);
  p += (size_t)kRangeListCap * kRangeThreads * 8;
  s.pair_y = reinterpret_cast<uint64_t*>(p);
  p += (size_t)kRangePairCap * 8;
  s.pair_q = reinterpret_cast<uint16_t*>(p);
  p += (size_t)kRangePairCap * 2;
  s.st_ids = reinterpret_cast<int32_t*>(p);
  s.sel = reinterpret_cast<uint32_t*>(p);
  p += (size_t)kKcapMax * 4;
  s.st_vals = reinterpret_cast<float*>(p);
  s.binlist = reinterpret_cast<BinMember*>(p);
  p += (size_t)kKcapMax * 4;
  s.hist = reinterpret_cast<uint32_t*>(p);
  p += (size_t)kSampleBins * 4;
  s.masks = reinterpret_cast<uint32_t*>(p);
  p += (size_t)mask_words * kRangeThreads * 4;
  s.tab = reinterpret_cast<RowEntry*>(p);
  p += (size_t)kRowsPerCta * sizeof(RowEntry);
  s.redo = reinterpret_cast<int32_t*>(p);
  p += (size_t)kRowsPerCta * 4;
  s.full = reinterpret_cast<uint64_t*>(p);
  s.empty = s.full + kRangeRingStages;
  s.sample_full = s.empty + kRangeRingStages;
  s.tau_full = s.sample_full + 2;
  s.cand_full = s.tau_full + 2;
  s.cand_free = s.cand_full + 1;
  p += 16 * 8;
  s.scan_f = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.scan_p = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.scan_a = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.ctl = reinterpret_cast<int*>(p);
  p += kRcWords * 4;
  s.hist_c = reinterpret_cast<uint32_t*>(p);
  s.sel_c = s.hist_c + kSampleBins / 32;
  return s;
}

// Position in the ring of the CTA's n-th copy (the producer and both consumer groups count the same
// sequence of copies): slot n mod NS, used for the (n / NS)-th time.  The sequence: the sample (stage 0) of
// the first live row; then for every live row the sample of the next live row (if there is one) followed
// by the row's own stages 0..S-1.  A slot's `empty` barrier sees every copy that goes through the slot, in
// order, and only the producer waits on it.  Its `full` barrier completes for row stages only and the two
// `sample_full` barriers for samples only, so that each is waited on by ONE group that takes its phases in
// order: a parity wait tells a phase only from its neighbours, and a group waiting on a barrier that also
// completes for the other group's copies would take one of those for its own.
struct RingPos {
  int slot;
  uint32_t use;
  __device__ __forceinline__ void step() {
    if (++slot == kRangeRingStages) {
      slot = 0;
      ++use;
    }
  }
  __device__ __forceinline__ void skip(int n) {
    for (int j = 0; j < n; ++j) step();
  }
};

// try_wait that may stay suspended in hardware for up to about `ns` nanoseconds before it reports "not yet"
// (it returns at once when the phase completes): a waiting warp then spends next to no issue slots on polling.
__device__ __forceinline__ bool mbar_try_wait_for(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}

// Bounded wait that also gives up when another role of the CTA has raised the abort flag.
__device__ __forceinline__ bool mbar_wait_abortable(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait_for(bar, parity, 4000u)) return true;
    if ((i & 7u) == 7u) {
      if (*abort_flag != 0) break;
      if (clock64() - t0 > kSpinCycles) break;
    }
  }
  return false;
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

// The same box asked into the L2 only, ahead of its copy: the ring's three stages cannot cover the latency of
// HBM under load (a stage comes back 3-4 K cycles after its slot was given up and is worked through in 1.3 K),
// the L2's they can.
__device__ __forceinline__ void tma_prefetch_box(const CUtensorMap* map, int x, int z) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(reinterpret_cast<uint64_t>(map)),
               "r"(x), "r"(0), "r"(z)
               : "memory");
}

// Histograms come in two levels: BINS fine bins and BINS / 32 coarse ones, coarse[c] counting what fine bins
// 32 c .. 32 c + 31 count (whoever adds to a fine bin adds to its coarse bin as well: shared-memory atomics
// that ask for no old value are cheap, a long search by one warp while the others wait is not).
//
// rank search: the largest bin b with (entries in bins > b) < target <= (entries in bins >= b), found by one
// warp with two short scans: over the coarse bins (lane 0 takes the topmost), then over the 32 fine bins of
// the coarse bin that holds the rank.  Every lane gets the result: bin + 1 in bits 0-11 of one word (0 when
// the histogram holds fewer than `target` entries) with the bin's own count in bits 12-31, and the count
// above the bin.  Counts stay below 2^20 (a row has at most 2^17 values).  With ZERO the warp also clears both
// levels (it must be the only reader).  Inlined on purpose, like everything on the roles' paths: an
// out-of-line function saves and restores registers through local memory, and local memory lies behind the
// ring's outstanding copies.
struct RankBin {
  uint32_t bin_count;  // (count << 12) | (bin + 1)
  uint32_t above;
  __device__ __forceinline__ int bin() const { return (int)(bin_count & 0xfffu) - 1; }
  __device__ __forceinline__ uint32_t count() const { return bin_count >> 12; }
};
__device__ __forceinline__ uint32_t warp_scan_incl(uint32_t v, int lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, v, d);
    if (lane >= d) v += n;
  }
  return v;
}
template <int BINS, bool ZERO>
__device__ __forceinline__ RankBin warp_rank_bin(uint32_t* fine, uint32_t* coarse, uint32_t target, int lane) {
  constexpr int C = BINS / 32;  // coarse bins
  constexpr int Q = C / 32;     // coarse bins per lane
  static_assert(BINS % 1024 == 0 && (Q == 1 || Q == 2), "1024 or 2048 bins");
  // lane l: coarse bins C - 1 - Q l (c_hi) and, with two to a lane, the one below it (c_lo)
  uint32_t c_hi, c_lo = 0;
  if (Q == 2) {
    const uint2 c = *reinterpret_cast<const uint2*>(coarse + C - 2 - 2 * lane);
    c_lo = c.x;
    c_hi = c.y;
  } else {
    c_hi = coarse[C - 1 - lane];
  }
  const uint32_t both = c_lo + c_hi;
  const uint32_t ab = warp_scan_incl(both, lane) - both;  // entries above this lane's upper coarse bin
  const bool in_hi = ab < target && target <= ab + c_hi;
  const bool in_lo = Q == 2 && ab + c_hi < target && target <= ab + both;
  const uint32_t votes = __ballot_sync(0xffffffffu, in_hi || in_lo);
  RankBin result{0u, 0u};
  if (votes != 0u) {
    const int l1 = __ffs((int)votes) - 1;
    // the coarse bin that holds the rank, and what lies above it
    const uint32_t mine = ((uint32_t)(C - 1 - Q * lane - (in_lo ? 1 : 0)) << 20) | (in_hi ? ab : ab + c_hi);
    const uint32_t got = __shfl_sync(0xffffffffu, mine, l1);
    const uint32_t cbin = got >> 20, above0 = got & 0xfffffu;
    const uint32_t f = fine[32u * cbin + 31u - (uint32_t)lane];  // lane 0 takes the topmost of its 32 fine bins
    const uint32_t ab2 = above0 + warp_scan_incl(f, lane) - f;
    const int l2 = __ffs((int)__ballot_sync(0xffffffffu, ab2 < target && target <= ab2 + f)) - 1;  // exists
    result.bin_count = (__shfl_sync(0xffffffffu, f, l2) << 12) | (32u * cbin + 31u - (uint32_t)l2 + 1u);
    result.above = __shfl_sync(0xffffffffu, ab2, l2);
  }
  if (ZERO) {
    __syncwarp();
    // a lane's share of the fine bins: BINS / 32 consecutive words; lanes start at different 16-byte pieces
    // so that the eight lanes served together touch eight different bank groups
    constexpr int P = BINS / 32;
    uint4* my = reinterpret_cast<uint4*>(fine + P * lane);
#pragma unroll
    for (int x = 0; x < P / 4; ++x) my[(x + lane) & (P / 4 - 1)] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int x = 0; x < Q; ++x) coarse[Q * lane + x] = 0u;
  }
  return result;
}

// ---------------------------------------------------------------------------------------------------
// what the three consumer roles share: how a thread finds its 64 bytes of a staged slice
// ---------------------------------------------------------------------------------------------------
template <int DTYPE, bool HAS_U>
struct StageReader {
  uint32_t my_row;  // this thread's 64 bytes inside a staged array
  uint32_t swz;     // 64-byte swizzle: 16-byte piece j sits at j ^ swz
  __device__ __forceinline__ explicit StageReader(int tid) : my_row((uint32_t)tid * 64u), swz(((uint32_t)tid >> 1) & 3u) {}
  // the j-th group of eight elements of this thread in the staged slice at `stage`
  __device__ __forceinline__ void load_group(uint32_t stage, int j, RawTile<DTYPE>& r) const {
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
  }
};

// ---------------------------------------------------------------------------------------------------
// sampler warps: tau0 of the NEXT row from its stage 0, while the filter warps stream the current row
// ---------------------------------------------------------------------------------------------------
// Threshold in two steps: maxima of groups of eight -> histogram by order-preserving key -> floor f with
// enough group maxima above it; linear histogram over [f, sample max] -> tau0.  Two ways through the second
// step:
//   * by group maxima (group_rank > 0, the usual case: the wanted rank m is a small fraction p = m / n of the
//     sample): with exchangeable entries a group of eight has its maximum above t with probability
//     1 - (1 - p(t))^8, so the value whose rank among the group maxima is g = n/8 (1 - (1 - p)^8) has rank m
//     among the elements on average.  Only the eight maxima a thread holds are binned again;
//   * by elements (group_rank == 0): the sample stays in registers as packed half-precision values between
//     the two steps and every value above f is binned.
// Either way the ring slot is given back as soon as the sample is in registers.  tau0 only steers how many
// candidates the filter keeps (the result is exact whatever it is; too few candidates send the row to the
// any-shape path), so neither the rounding to 11 bits nor the translation of the rank costs exactness.
// Sampler thread t looks after ranges t, t + NT, t + 2 NT, ... (NT sampler threads; the last round may be short).
//
// FIRST = true is the same work done once, for the CTA's first row, by the finisher warps (which have nothing
// to do yet): many more threads, so the first threshold - which the whole CTA waits for - comes sooner; the
// sampler warps proper (FIRST = false) start on the second row at the same time.  The two work side by
// side, so the first-row instance has a histogram (the finisher's bins) and control words of its own.
template <int DTYPE, bool HAS_U, bool HAS_T, bool BY_GROUPS, int NA, int BAR_A, bool FIRST>
__device__ __forceinline__ void range_sampler_role(const RowArgs& a, const RangeCfg& cfg, const RangeSmem& sm, int tid) {
  constexpr int NT_A = NA * 32;
  constexpr int kBin = FIRST ? kRcBBin : kRcABin, kSmaxKey = FIRST ? kRcBSmaxKey : kRcSmaxKey;
  uint32_t* const hist = FIRST ? sm.sel : sm.hist;
  uint32_t* const hist_c = FIRST ? sm.sel_c : sm.hist_c;
  // An atomic with some lanes switched off runs several times slower than one with all lanes on, and lanes that
  // hit the same word cost nothing extra when the old value is not asked for: a lane with nothing to count
  // adds to a word nobody reads.
  uint32_t* const trash = reinterpret_cast<uint32_t*>(sm.ctl + (FIRST ? kRcTrashB : kRcTrashA));
  constexpr int TI = DTYPE != 0 ? 4 : 2;                     // groups of eight elements per range in stage 0
  constexpr int NR = (kRangeThreads + NT_A - 1) / NT_A;       // ranges per sampler thread (at most)
  constexpr int NG = NR * TI;                                 // groups per sampler thread (at most)
  const int lane = tid & 31, warp_a = tid >> 5;
  const float neg_inf = __int_as_float(0xff800000);
  const float lowest = -3.402823466e38f;  // with this threshold every finite value is a candidate
  volatile int* abort_flag = sm.ctl + kRcAbort;
  const uint64_t s2 = pack2(a.s, a.s), t2 = pack2(a.inv_T, a.inv_T);
  const uint32_t ring_addr = smem_u32(sm.ring);
  const uint32_t n_live = (uint32_t)sm.ctl[kRcLive];
  const uint32_t rank = (uint32_t)(BY_GROUPS ? cfg.group_rank : cfg.sample_rank);
  RingPos pos{0, 0};
  if (!FIRST) pos.step();  // the second row's sample is the CTA's second copy
  for (uint32_t k = FIRST ? 0u : 1u; k < (FIRST ? min(n_live, 1u) : n_live); ++k) {  // live rows of this CTA
    SJD_PHASE_BEGIN();
    // ---------------- the sample into registers; first pass on the way: maxima of groups of eight, by key ----------------
    const bool ok = mbar_wait_abortable(&sm.sample_full[k & 1u], (k >> 1) & 1u, abort_flag);
    SJD_PHASE(0);
    __half2 cache[BY_GROUPS ? 1 : NG * 4];
    float gmax[NG];
    float smax = neg_inf;
    // (rounds in which none of a warp's threads has a range leave their entries as they are: nothing)
#pragma unroll
    for (int g = 0; g < NG; ++g) gmax[g] = neg_inf;
#pragma unroll
    for (int x = 0; x < (BY_GROUPS ? 1 : NG * 4); ++x) cache[x] = __floats2half2_rn(neg_inf, neg_inf);
    if (ok) {
      const uint32_t stage0 = ring_addr + (uint32_t)pos.slot * (2 * kRangeStageBytes);
      // one group of eight per round.  The loop is kept rolled (the code of all roles has to stay in the
      // instruction cache): what a round finds is pushed in at the front of gmax / cache, the older entries move up.
#pragma unroll 1
      for (int g = 0; g < NG; ++g) {
        const int r = g / TI, j = g % TI;
        if (warp_a * 32 + r * NT_A >= kRangeThreads) continue;  // none of this warp's threads has a range in this round
        // a thread without a range in the last round works on a copy of range 255 and counts nothing (the
        // warp stays together for the vote below)
        const bool have = tid + r * NT_A < kRangeThreads;
        const StageReader<DTYPE, HAS_U> rd(have ? tid + r * NT_A : kRangeThreads - 1);
#pragma unroll
        for (int x = NG - 1; x >= 1; --x) gmax[x] = gmax[x - 1];
        if (!BY_GROUPS) {
#pragma unroll
          for (int x = NG * 4 - 1; x >= 4; --x) cache[BY_GROUPS ? 0 : x] = cache[BY_GROUPS ? 0 : x - 4];
        }
        RawTile<DTYPE> raw;
        rd.load_group(stage0, j, raw);
        float y[8];
        merge_raw<DTYPE, HAS_U, HAS_T>(raw, s2, t2, y);
        float m8 = canonical(max3(max3(max3(neg_inf, y[0], y[1]), y[2], y[3]), max3(y[4], y[5], y[6]), y[7]));
        if (!have) m8 = neg_inf;
        gmax[0] = m8;
        if (!BY_GROUPS) {
#pragma unroll
          for (int q = 0; q < 8; ++q) y[q] = have ? canonical(y[q]) : neg_inf;
#pragma unroll
          for (int q = 0; q < 4; ++q) cache[BY_GROUPS ? 0 : q] = __floats2half2_rn(y[2 * q], y[2 * q + 1]);
        }
        if (!BY_GROUPS && cfg.sample_all) {
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const uint32_t bin = float_key(y[q]) >> kSampleKeyShift;
            atomicAdd(have ? &hist[bin] : trash, 1u);
            atomicAdd(have ? &hist_c[bin >> 5] : trash, 1u);
          }
        } else {
          // group maxima crowd into a few coarse bins: lanes that meet in one cost no more than lanes apart
          const uint32_t bin = float_key(m8) >> kSampleKeyShift;
          atomicAdd(have ? &hist[bin] : trash, 1u);
          atomicAdd(have ? &hist_c[bin >> 5] : trash, 1u);
        }
        smax = fmaxf(smax, m8);
      }
    }
    if (NA <= 8) {
      __syncwarp();
      if (lane == 0) {
        // the slot's barrier counts eight warps: the sampler's share them out
        const int share = 8 / NA + (warp_a < 8 % NA ? 1 : 0);
        mbar_arrive(&sm.empty[pos.slot], (uint32_t)share);
      }
    } else {
      group_sync<NT_A, BAR_A>();
      if (tid == 0) mbar_arrive(&sm.empty[pos.slot], 8u);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, d));
    if (lane == 0) atomicMax(reinterpret_cast<unsigned int*>(&sm.ctl[kSmaxKey]), float_key(smax));
    if (group_any<NT_A, BAR_A>(!ok)) {
      if (tid == 0) *abort_flag = 1;
      return;
    }
    SJD_PHASE(1);
    // at least `rank` group maxima (or, binning everything, elements) are >= the lower edge of this bin.  One
    // warp searches and clears the histogram; the others wait.
    if (warp_a == 0) {
      const RankBin rb = warp_rank_bin<kSampleBins, true>(hist, hist_c, rank, lane);
      if (lane == 0) sm.ctl[kBin] = rb.bin();
    }
    group_sync<NT_A, BAR_A>();
    SJD_PHASE(2);
    const int cbin = sm.ctl[kBin];
    float floor_y = cbin >= 0 ? key_float((uint32_t)cbin << kSampleKeyShift) : lowest;
    if (!(floor_y >= lowest)) floor_y = lowest;  // edge fell on -inf or into the NaN patterns
    const float top_y = key_float((uint32_t)sm.ctl[kSmaxKey]);
    const bool refine = floor_y > lowest && top_y >= floor_y && top_y <= 3.402823466e38f;
    const float range = __fsub_rn(top_y, floor_y);
    const float scale = (refine && range > 0.0f) ? __fdiv_rn((float)kSampleBins - 0.5f, range) : 0.0f;
    // ---------------- second pass: linear bins over [floor, sample max] ----------------
    float tau0 = lowest;
    if (refine) {
      if (BY_GROUPS) {
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          const int bin = min(max(__float2int_rd(__fmul_rn(__fsub_rn(gmax[g], floor_y), scale)), 0), kSampleBins - 1);
          atomicAdd(gmax[g] >= floor_y ? &hist[bin] : trash, 1u);
          atomicAdd(gmax[g] >= floor_y ? &hist_c[bin >> 5] : trash, 1u);
        }
      } else {
#pragma unroll
        for (int j = 0; j < (BY_GROUPS ? 0 : NG * 4); ++j) {
          const float2 v = __half22float2(cache[j]);
          const int b0 = min(max(__float2int_rd(__fmul_rn(__fsub_rn(v.x, floor_y), scale)), 0), kSampleBins - 1);
          const int b1 = min(max(__float2int_rd(__fmul_rn(__fsub_rn(v.y, floor_y), scale)), 0), kSampleBins - 1);
          atomicAdd(v.x >= floor_y ? &hist[b0] : trash, 1u);
          atomicAdd(v.x >= floor_y ? &hist_c[b0 >> 5] : trash, 1u);
          atomicAdd(v.y >= floor_y ? &hist[b1] : trash, 1u);
          atomicAdd(v.y >= floor_y ? &hist_c[b1 >> 5] : trash, 1u);
        }
      }
      group_sync<NT_A, BAR_A>();
      SJD_PHASE(3);
      if (warp_a == 0) {
        const int fbin = warp_rank_bin<kSampleBins, true>(hist, hist_c, rank, lane).bin();
        if (fbin > 0 && scale > 0.0f) {
          // a little below the lower edge of the bin, so that rounding cannot exclude one of its members
          const float t = __fmul_rd(__fdiv_rd((float)fbin, scale), 0.99999f);
          tau0 = __fadd_rd(floor_y, t);
        } else if (fbin >= 0) {
          tau0 = floor_y;
        }
      }
    } else {
      group_sync<NT_A, BAR_A>();  // every thread has read kRcSmaxKey before it is reset below
    }
    // a word of its own for each of four consecutive rows: the filter reads it at the start of the row, and
    // the ring keeps the sampler less than two rows ahead of the filter
    if (tid == 0) {
      sm.ctl[kSmaxKey] = 0;  // every thread has read it (barrier above)
      sm.ctl[kRcTau0 + (int)(k & 3u)] = __float_as_int(tau0);
      sm.ctl[kRcTop0 + (int)(k & 3u)] = __float_as_int(top_y);
      mbar_arrive(&sm.tau_full[k & 1u]);
    }
    group_sync<NT_A, BAR_A>();  // the histogram is clear and kRcSmaxKey reset before the next row's first pass
    SJD_PHASE(4);
    // sample(k+1) follows sample(k) after the S stages of row k-1 and itself (k >= 1)
    pos.skip(1 + cfg.stages);
  }
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
  const int lane = tid & 31;
  const int mask_words = cfg.mask_words;
  volatile int* abort_flag = sm.ctl + kRcAbort;
  const uint64_t s2 = pack2(a.s, a.s), t2 = pack2(a.inv_T, a.inv_T);
  const uint32_t ring_addr = smem_u32(sm.ring);
  const StageReader<DTYPE, HAS_U> rd(tid);
  const uint32_t list_base = smem_u32(sm.ylist) + (uint32_t)tid * 8u;
  const uint32_t list_limit = list_base + (uint32_t)(kRangeListCap - 4) * kStride;  // beyond it a group may not fit
  const uint32_t n_live = (uint32_t)sm.ctl[kRcLive];
  RingPos pos{0, 0};
  pos.step();  // the CTA's first copy is the first row's sample
  uint32_t full_phase = 0;  // bit s: parity of the next phase of full[s] this group waits for
  int flip = 0;
  for (uint32_t k = 0; k < n_live; ++k) {  // live rows of this CTA
    // from the CTA's last row on, the verification grid may be scheduled (it waits for this grid's end)
    if (k + 1 == n_live) allow_dependent_launch();
    else pos.step();  // the next row's sample comes before this row's stages
    SJD_PHASE_BEGIN();
    bool ok = mbar_wait_abortable(&sm.tau_full[k & 1u], (k >> 1) & 1u, abort_flag);
    SJD_PHASE(8);
    const float tau0 = __int_as_float(sm.ctl[kRcTau0 + (int)(k & 3u)]);
    const int top_bits = sm.ctl[kRcTop0 + (int)(k & 3u)];

    uint32_t cur = list_base;  // shared-memory address of the thread's next free entry
    uint32_t imw = 0;          // inverted hit bits of the groups filtered since the last full mask word
    bool overflow = false;
    // One group: four pairs.  A pair is stored at the cursor, and the cursor moves on, only for a hit, i.e.
    // when max(pair) >= thr.  A pair of NaNs and -inf never hit.
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
      for (int q = 0; q < 4; ++q) {
        const float m = fmaxf(y[2 * q], y[2 * q + 1]);
        // hit: the pair is stored and the cursor moves on; miss: the pair's bit is set in the inverted mask
        // (all predicated, no branch).  A store with no lane on costs shared memory nothing, one with two or
        // three lanes on one pass instead of the two a full warp's 256 bytes take.
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ge.f32 p, %2, %3;\n\t@p st.shared.v2.f32 [%0], {%6, %7};\n\t@p add.u32 %0, %0, %4;\n\t"
            "@!p or.b32 %1, %1, %5;\n\t}"
            : "+r"(d), "+r"(imw)
            : "f"(m), "f"(thr), "r"(kStride), "r"(8u >> q), "f"(y[2 * q]), "f"(y[2 * q + 1])
            : "memory");
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
    // ---------------- the row against tau0 ----------------
    for (int s = 0; s < cfg.stages; ++s) {
      if (ok) ok = mbar_wait_abortable(&sm.full[pos.slot], (full_phase >> pos.slot) & 1u, abort_flag);
      full_phase ^= 1u << pos.slot;
      if (ok) {
        const uint32_t stage = ring_addr + (uint32_t)pos.slot * (2 * kRangeStageBytes);
        RawTile<DTYPE> raw[TI];
#pragma unroll
        for (int j = 0; j < TI; ++j) rd.load_group(stage, j, raw[j]);
#pragma unroll
        for (int j = 0; j < TI; ++j) filter_group(raw[j], tau0);
        end_stage(s);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[pos.slot]);
      pos.step();
    }
    SJD_PHASE(9);
    // ---------------- drain: this thread's list becomes its run of the pair list ----------------
    // Threads own ascending id ranges and meet their ids in ascending order, so writing the runs one
    // after the other yields the candidate pairs in ascending id order.  A pair goes over as it is; the
    // finisher sorts out which of its two values reach tau0.
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
    // the pair list must be back from the finisher
    if (ok && k > 0) ok = mbar_wait_abortable(sm.cand_free, (k - 1) & 1u, abort_flag);
    SJD_PHASE(10);
    // one scan carries the entry counts (bits 0-13: at most 35 each) and the number of threads whose list ran
    // over (bits 14-22) or whose wait gave up (bits 23-31)
    uint32_t sum;
    const uint32_t mine = (uint32_t)n_e | (overflow ? 1u << 14 : 0u) | (ok ? 0u : 1u << 23);
    const uint32_t my_off = group_scan1<NT_F, BAR_F, uint32_t>(mine, tid, sm.scan_f, flip, &sum) & 0x3fffu;
    if ((sum >> 23) != 0u) {
      if (tid == 0) *abort_flag = 1;
      return;  // the row is not handed over: the finisher's wait ends on the flag and it marks the rows
    }
    const uint32_t n_pairs = sum & 0x3fffu;
    // a list that ran over, or more pairs than the finisher holds: it redoes the row by the any-shape path
    const bool fallback = ((sum >> 14) & 0x1ffu) != 0u || n_pairs > (uint32_t)kRangePairCap;
    SJD_PHASE(11);
    if (!fallback) {
      // (1) the pairs, four at a time: loads and stores of different entries do not wait for one another
      uint32_t y_at = smem_u32(sm.pair_y) + my_off * 8u;
      for (int e0 = 0; e0 < n_e; e0 += 4) {
        uint64_t v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)  // entries past n_e are read (inside the list) and dropped
          asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v[u]) : "r"(list_base + (uint32_t)min(e0 + u, kRangeListCap - 1) * kStride));
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (e0 + u < n_e) asm volatile("st.shared.b64 [%0], %1;" ::"r"(y_at + 8u * (uint32_t)u), "l"(v[u]) : "memory");
        }
        y_at += 32u;
      }
      // (2) their pair numbers: the set hit bits, word by word.  The walk over the words is the same for
      // every thread of the warp (one mask load per word, outside the inner loop); only the number of bits
      // in a word differs from lane to lane.  (With the word change inside a per-entry loop every entry paid
      // for a divergent branch and a shared-memory load: the drain took three times as long.)
      uint32_t q_at = smem_u32(sm.pair_q) + my_off * 2u;
      uint32_t qn = (uint32_t)(tid * (cfg.range_len >> 1));  // pair number of the first bit of the current mask word
      for (int w = 0; w < mask_words; ++w) {
        uint32_t x = ~sm.masks[(size_t)w * NT_F + tid];
        while (x != 0u) {
          const uint32_t bitpos = (uint32_t)__clz((int)x);
          x &= ~(0x80000000u >> bitpos);
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(q_at), "h"((uint16_t)(qn + bitpos)) : "memory");
          q_at += 2u;
        }
        qn += 32u;
      }
    }
    if (tid == 0) {
      sm.ctl[kRcRowTau0] = __float_as_int(tau0);
      sm.ctl[kRcRowTop] = top_bits;
      sm.ctl[kRcRowPairs] = (int)n_pairs;
      sm.ctl[kRcRowFallback] = fallback ? 1 : 0;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(sm.cand_full);
    SJD_PHASE(12);
  }
}

// ---------------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------------
template <int DTYPE, int NP, int NA, bool HAS_U, bool HAS_T, bool BY_GROUPS>
__global__ void __launch_bounds__((8 + NP + NA + 1) * 32, 1)
rows_ranges_kernel(const RowArgs a, const RangeCfg cfg, const __grid_constant__ CUtensorMap map_c,
                   const __grid_constant__ CUtensorMap map_u) {
  constexpr int NF = 8;
  constexpr int NT_F = kRangeThreads, NT_P = NP * 32;
  constexpr int BAR_P = 2;  // named barrier of the finisher warps (the filter warps use 1, the sampler warps 3)
  constexpr int kFinItems = kKcapMax / NT_P;                        // staged survivors per finisher thread
  constexpr int kPairChunk = (kRangePairCap + NT_P - 1) / NT_P;     // candidate pairs per finisher thread
  constexpr int NS = kRangeRingStages;
  constexpr int BW = 64 / (DTYPE != 0 ? 2 : 4);  // elements per stage and range
  static_assert(NT_F == NF * 32 && kFinItems * NT_P == kKcapMax && (kFinItems == 4 || kFinItems == 8), "group sizes");
  static_assert(2 * kPairChunk <= 32 && NP <= 16 && (NP & (NP - 1)) == 0, "hit bits in one word; warp maxima in the spare scratch slots");
  extern __shared__ unsigned char smem_raw[];
  RangeSmem sm = carve_range_smem(smem_raw, cfg.mask_words);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool has_u = HAS_U;  // the host picks the instantiation: uncond given, 1/T != 1, thresholds by group maxima
  const float neg_inf = __int_as_float(0xff800000);

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], NF);
    }
    for (int p = 0; p < 2; ++p) {
      mbar_init(&sm.sample_full[p], 1);
      mbar_init(&sm.tau_full[p], 1);
    }
    mbar_init(sm.cand_full, NF);  // every filter warp arrives when its share of the pair list is written
    mbar_init(sm.cand_free, NP);  // every finisher warp arrives when its share is in registers
    for (int k = 0; k < kRcWords; ++k) sm.ctl[k] = 0;
    fence_barrier_init();
  }
  for (int j = threadIdx.x; j < kSampleBins; j += blockDim.x) sm.hist[j] = 0;
  for (int j = threadIdx.x; j < kSelBins; j += blockDim.x) sm.sel[j] = 0;
  for (int j = threadIdx.x; j < kSampleBins / 32 + kSelBins / 32; j += blockDim.x) sm.hist_c[j] = 0;  // both coarse levels
  // everything above touched shared memory only; global memory is read and written from here on, so a
  // launch that was allowed to overlap the previous kernel of the stream waits for that kernel's end here
  grid_dependency_wait();
  __syncthreads();
  // ---- the CTA's rows: row_begin + blockIdx.x, + gridDim.x, ... (at most kRowsPerCta of them inside
  // [row_begin, row_end), which the host guarantees).  Rows beyond their sequence's window length have no
  // logits to look at and get their empty result here; the others go into a table with everything the roles
  // need to know about them, so that no role reads global memory at a row boundary (behind the ring's
  // outstanding copies such a load takes thousands of cycles).
  if (warp == 0) {
    const int row = cfg.row_begin + (int)blockIdx.x + lane * (int)gridDim.x;
    bool live = false;
    RowEntry e{row, 0, 0, -1};
    if (row < cfg.row_end) {
      const int b = row / a.W, i = row - b * a.W;
      const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
      live = i < L;
      if (live) {
        e.pos = (a.pos_base ? a.pos_base[b] : 0) + i;
        e.iter = a.iteration ? a.iteration[b] : a.iteration0;
        e.draft = a.drafts ? a.drafts[row] : -1;
      } else {
        a.out_cnt[row] = 0;
        a.scratch[row] = RowScratch{0.0f, -1, 0.0f, 0};
      }
    }
    const uint32_t votes = __ballot_sync(0xffffffffu, live);
    if (live) sm.tab[__popc(votes & ((1u << lane) - 1u))] = e;
    if (lane == 0) sm.ctl[kRcLive] = __popc(votes);
  }
  __syncthreads();
  volatile int* abort_flag = sm.ctl + kRcAbort;
  const int n_live = sm.ctl[kRcLive];

  if (warp == NF + NP + NA) {
    // ====================================== producer warp ======================================
    if (lane != 0) return;
    RingPos pos{0, 0};
    bool ok = true;
    const uint32_t stage_bytes = (uint32_t)kRangeStageBytes * (has_u ? 2u : 1u);
    // per slot, as bit masks (arrays indexed by the slot would live in local memory): the parity of the next
    // row-stage phase of full[slot]; whether the latest copy into the slot was a sample, and that copy's parity
    uint32_t stage_parity = 0, last_is_sample = 0, last_parity = 0, used = 0;
    int last_sample_of = 0;
    auto issue = [&](int x, int row, int sample_of) {  // sample_of: -1 for a row stage, else the live row's index
      if (pos.use > 0) ok = mbar_wait_abortable(&sm.empty[pos.slot], (pos.use - 1) & 1u, abort_flag);
      ok = ok && (*abort_flag == 0);
      if (!ok) return;
      unsigned char* dst = sm.ring + (size_t)pos.slot * (2 * kRangeStageBytes);
      const uint32_t bit = 1u << pos.slot;
      uint64_t* bar;
      uint32_t parity;
      if (sample_of >= 0) {
        bar = &sm.sample_full[sample_of & 1];
        parity = ((uint32_t)sample_of >> 1) & 1u;
        last_is_sample |= bit;
        last_sample_of = sample_of;
      } else {
        bar = &sm.full[pos.slot];
        parity = (stage_parity >> pos.slot) & 1u;
        stage_parity ^= bit;
        last_is_sample &= ~bit;
      }
      last_parity = parity ? (last_parity | bit) : (last_parity & ~bit);
      used |= bit;
#ifdef SJD_TEST_DROP_COPY
      // test builds only: the CTA's copy number SJD_TEST_DROP_COPY is never issued, so that the wait for it
      // runs out and the time-out path (status instead of a hang) can be watched
      if ((int)(pos.use * NS + pos.slot) == SJD_TEST_DROP_COPY) {
        used &= ~bit;
        pos.step();
        return;
      }
#endif
      mbar_arrive_expect_tx(bar, stage_bytes);
      tma_load_box(dst, &map_c, x, row, bar);
      if (has_u) tma_load_box(dst + kRangeStageBytes, &map_u, x, row, bar);
      pos.step();
    };
    auto prefetch = [&](int x, int row) {
      tma_prefetch_box(&map_c, x, row);
      if (has_u) tma_prefetch_box(&map_u, x, row);
    };
    if (n_live > 0) {
      issue(0, sm.tab[0].row, 0);
    }
    for (int k = 0; k < n_live && ok; ++k) {
      if (k + 1 < n_live) issue(0, sm.tab[k + 1].row, k + 1);
      const int row = sm.tab[k].row;
      for (int s = 0; s < cfg.stages && ok; ++s) {
        // the stage that will take this stage's slot next is asked into the L2 now (stage 0 of a row comes
        // with that row's sample)
        {
          const int ahead = s + NS;
          if (ahead < cfg.stages) prefetch(ahead * BW, row);
          else if (k + 1 < n_live && ahead - cfg.stages > 0 && ahead - cfg.stages < cfg.stages) prefetch((ahead - cfg.stages) * BW, sm.tab[k + 1].row);
        }
        issue(s * BW, row, -1);
      }
    }
    // drain: every copy armed here must have landed before the CTA may exit.  The latest copy into a slot
    // is the only one that can still be in flight; a slot whose latest copy was a sample holds the latest
    // sample issued (two samples are at least three copies apart).
#pragma unroll
    for (int sl = 0; sl < NS; ++sl) {
      if ((used >> sl) & 1u) {
        uint64_t* bar = ((last_is_sample >> sl) & 1u) ? &sm.sample_full[last_sample_of & 1] : &sm.full[sl];
        mbar_wait(bar, (last_parity >> sl) & 1u);
      }
    }
    if (!ok) *abort_flag = 1;
    return;
  }

  if (warp < NF) {
    // ======================================= filter warps =======================================
    range_filter_role<DTYPE, HAS_U, HAS_T>(a, cfg, sm, threadIdx.x);
    return;
  }
  if (warp >= NF + NP) {
    // ======================================= sampler warps =======================================
    range_sampler_role<DTYPE, HAS_U, HAS_T, BY_GROUPS, NA, 3, false>(a, cfg, sm, threadIdx.x - (NF + NP) * 32);
    return;
  }

  // ======================================= finisher warps =======================================
  const int tid = threadIdx.x - NT_F;  // 0 .. NT_P-1
  // the first row's threshold, while there is nothing to finish yet
  range_sampler_role<DTYPE, HAS_U, HAS_T, BY_GROUPS, NP, BAR_P, true>(a, cfg, sm, tid);
  int flip = 0;
  bool dead = false;
  for (int k = 0; k < n_live; ++k) {
    // from the CTA's last row on, the verification grid may be scheduled (it waits for this grid's end)
    if (k + 1 == n_live) allow_dependent_launch();
    SJD_PHASE_BEGIN();
    const RowEntry re = sm.tab[k];
    const int row = re.row, draft = re.draft;
    const int b = row / a.W;
    RowScratch* rs = a.scratch + row;
    const int kcap = a.kcap;
    // the row's own random number: needed last, computed by one thread while the others wait
    if (tid == NT_P - 1) {
      const uint64_t r = random64(philox4x32_10((uint32_t)re.pos, (uint32_t)(a.seq_base + b), (uint32_t)re.iter,
                                                (uint32_t)a.purpose, a.seed_lo, a.seed_hi));
      sm.ctl[kRcRndLo] = (int)(uint32_t)r;
      sm.ctl[kRcRndHi] = (int)(uint32_t)(r >> 32);
    }
    if (!dead) dead = !mbar_wait_abortable(sm.cand_full, (uint32_t)k & 1u, abort_flag);
    dead = group_any<NT_P, BAR_P>(dead || (*abort_flag != 0));
    if (dead) {
      if (tid == 0) {
        *abort_flag = 1;
        a.out_cnt[row] = 0;
        *rs = RowScratch{0.0f, -1, 0.0f, kRowStatusTimeout};
      }
      continue;
    }
    SJD_PHASE(16);
    const float tau0 = __int_as_float(sm.ctl[kRcRowTau0]);
    const float top = __int_as_float(sm.ctl[kRcRowTop]);
    const uint32_t n_pairs = (uint32_t)sm.ctl[kRcRowPairs];
    bool fallback = kcap > kKcapMax || sm.ctl[kRcRowFallback] != 0;
    // ---- every thread takes an equal share of the pair list into registers: a run of consecutive pairs, so
    // that concatenating the threads' survivors keeps the id order.  The list then goes straight back to the
    // filter warps, which may already be waiting to write the next row's.
    // The shares differ by one pair at most (the first n mod NT threads take one more), and a warp skips the
    // slots none of its threads fills: with 2,600 pairs most warps work on five slots, not on all seven.
    const uint32_t share = fallback ? 0u : n_pairs / NT_P, extra = fallback ? 0u : n_pairs % NT_P;
    const uint32_t my_first = (uint32_t)tid * share + min((uint32_t)tid, extra);
    const uint32_t my_count = share + ((uint32_t)tid < extra ? 1u : 0u);          // <= kPairChunk
    const uint32_t wcount = share + (((uint32_t)tid & ~31u) < extra ? 1u : 0u);  // the warp's largest share
    float2 v[kPairChunk];
    uint32_t qq[(kPairChunk + 1) / 2];  // pair numbers, two to a word
#pragma unroll
    for (int j = 0; j < (kPairChunk + 1) / 2; ++j) qq[j] = 0u;
#pragma unroll
    for (int j = 0; j < kPairChunk; ++j) {
      if ((uint32_t)j < wcount) {
        // a slot beyond the thread's share reads another pair of this row (the next thread's, or the row's
        // last) and is masked out below - except for the row's maximum, which it cannot raise
        const uint32_t at = min(my_first + (uint32_t)j, n_pairs - 1u);  // wcount > 0, so the row has pairs
        v[j] = *reinterpret_cast<const float2*>(&sm.pair_y[at]);
        const uint32_t q = sm.pair_q[at];
        if ((j & 1) == 0) qq[j >> 1] = q;
        else qq[j >> 1] |= q << 16;
      }
    }
    if (tid == 0) {
      sm.ctl[kRcGather] = 0;
      sm.ctl[kRcPtok] = 0;
      sm.ctl[kRcFoundId] = -1;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(sm.cand_free);
    if (fallback) {
      if (tid == 0) sm.redo[sm.ctl[kRcRedo]++] = row;  // redone by the any-shape path after the last row
      continue;
    }
    // ---- linear bins 1 .. kSelBins - 1 over [tau0, top] (top: the largest sample value; anything above it
    // lands in the last bin); monotone in y, so a higher bin never holds a smaller value.  Bin 0 takes what is
    // no candidate (below tau0, NaN, a slot beyond the thread's share): every lane of every update is on (a
    // partly switched-off atomic is several times slower, lanes that meet in one word cost nothing) and no
    // address has to be chosen.  A thread keeps the bins of its values in registers.
    const float range = __fsub_rn(top, tau0);
    const float scale = range > 0.0f ? __fdiv_rn((float)(kSelBins - 1) * 0.999f, range) : 0.0f;
    uint32_t code[kPairChunk];
    float vmax = neg_inf;
#pragma unroll
    for (int j = 0; j < kPairChunk; ++j) {
      if ((uint32_t)j >= wcount) continue;
      const bool mine = (uint32_t)j < my_count;
      const bool v0 = mine && v[j].x >= tau0, v1 = mine && v[j].y >= tau0;  // false for NaN
      const int q0 = min(__float2int_rd(__fmul_rn(__fsub_rn(v[j].x, tau0), scale)), kSelBins - 2);
      const int q1 = min(__float2int_rd(__fmul_rn(__fsub_rn(v[j].y, tau0), scale)), kSelBins - 2);
      const uint32_t c0 = v0 ? (uint32_t)q0 + 1u : 0u, c1 = v1 ? (uint32_t)q1 + 1u : 0u;
      code[j] = c0 | (c1 << 16);
      // the largest candidate is the largest value of the list (a NaN is passed over, a value below tau0
      // lies below every candidate, and a row without candidates is redone anyway)
      vmax = max3(vmax, v[j].x, v[j].y);
      atomicAdd(&sm.sel[c0], 1u);
      atomicAdd(&sm.sel_c[c0 >> 5], 1u);
      atomicAdd(&sm.sel[c1], 1u);
      atomicAdd(&sm.sel_c[c1 >> 5], 1u);
    }
    // the row's maximum: per warp here, combined after the barrier
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, d));
    float* const warp_max = reinterpret_cast<float*>(sm.scan_p + 64);
    if (lane == 0) warp_max[warp - NF] = vmax;
    group_sync<NT_P, BAR_P>();
    SJD_PHASE(17);
    // ---- exact K-th largest: threshold bin, then ranking inside it by (y descending, id ascending).  Every
    // warp searches the histogram for itself (the search is short, a barrier would cost more).
    const RankBin rb = warp_rank_bin<kSelBins, false>(sm.sel, sm.sel_c, (uint32_t)kcap, lane);
    const int tbin = rb.bin();
    const int need = kcap - (int)rb.above;  // members of the threshold bin that survive
    const int nbin = (int)rb.count();
    // lane l takes warp (l mod NP)'s maximum; the butterfly leaves the row's maximum in every lane
    vmax = warp_max[lane & (NP - 1)];
#pragma unroll
    for (int d = NP / 2; d > 0; d >>= 1) vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, d));
    // fewer than kcap candidates (the sampled threshold was too high), a threshold bin too crowded for the
    // on-chip ranking, or no finite maximum: the any-shape path redoes the row
    if (tbin <= 0 || nbin > kBinListCap || !(vmax <= 3.402823466e38f)) fallback = true;  // bin 0: the rank lies among what is no candidate
    SJD_PHASE(18);
    const uint32_t tcode = (uint32_t)tbin;  // a value's code is its bin
    uint32_t above = 0;  // bit 2j + h: value h of pair j lies in a bin above the threshold bin
    uint32_t hits = 0;   // likewise: it lies in the threshold bin
    int my_at0 = -1, my_at1 = -1;
    bool many = false;
    if (!fallback) {
#pragma unroll
      for (int j = 0; j < kPairChunk; ++j) {
        if ((uint32_t)j >= wcount) continue;
        const uint32_t c0 = code[j] & 0xffffu, c1 = code[j] >> 16;
        above |= (c0 > tcode ? 1u : 0u) << (2 * j);
        above |= (c1 > tcode ? 1u : 0u) << (2 * j + 1);
        hits |= (c0 == tcode ? 1u : 0u) << (2 * j);
        hits |= (c1 == tcode ? 1u : 0u) << (2 * j + 1);
      }
      // the members of the threshold bin (a handful per row) go on a list: value and position in the pair
      // list; the thread remembers where its first two went
      if (hits != 0u) {
#pragma unroll
      for (int j = 0; j < kPairChunk; ++j) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if ((hits >> (2 * j + h)) & 1u) {
            const int at = atomicAdd(&sm.ctl[kRcGather], 1);
            sm.binlist[at] = BinMember{h == 0 ? v[j].x : v[j].y, (int)(2u * (my_first + j)) + h};
            if (my_at0 < 0) my_at0 = at;
            else if (my_at1 < 0) my_at1 = at;
            else many = true;
          }
        }
      }
      }
    }
    group_sync<NT_P, BAR_P>();
    // one warp per member ranks it against the list, a lane per rival: the `need` best survive (ties to the
    // lower id), the others are marked (slot made negative)
    if (!fallback) {
      for (int x = warp - NF; x < nbin; x += NP) {
        const BinMember me = sm.binlist[x];  // only this warp marks member x, and only below
        int ahead = 0;
        for (int z = lane; z < nbin; z += 32) {
          const BinMember o = sm.binlist[z];
          const int o_slot = o.slot < 0 ? -1 - o.slot : o.slot;  // another warp may have marked it already
          ahead += (o.y > me.y || (o.y == me.y && o_slot < me.slot)) ? 1 : 0;
        }
        const int rank = __reduce_add_sync(0xffffffffu, ahead);
        if (lane == 0 && rank >= need) sm.binlist[x].slot = -1 - me.slot;
      }
    }
    group_sync<NT_P, BAR_P>();
    // every thread strikes its marked members from `hits`
    if (!fallback && hits != 0u) {
      const int slot0 = (int)(2u * my_first);
      if (!many) {
        if (my_at0 >= 0) {
          const int sl = sm.binlist[my_at0].slot;
          if (sl < 0) hits &= ~(1u << (-1 - sl - slot0));
        }
        if (my_at1 >= 0) {
          const int sl = sm.binlist[my_at1].slot;
          if (sl < 0) hits &= ~(1u << (-1 - sl - slot0));
        }
      } else {  // more than two members in one thread's share (many equal values): look through the list
        for (int x = 0; x < nbin; ++x) {
          const int sl = sm.binlist[x].slot;
          const uint32_t rel = (uint32_t)(-1 - sl - slot0);
          if (sl < 0 && rel < 2u * my_count) hits &= ~(1u << rel);
        }
      }
    }
    SJD_PHASE(19);
    uint32_t total_alive;
    uint32_t out_pos = group_scan1<NT_P, BAR_P, uint32_t>((uint32_t)__popc(above | hits), tid, sm.scan_p, flip, &total_alive);
    if (!fallback && total_alive != (uint32_t)kcap) fallback = true;  // cannot happen; keep the result exact anyway
    if (!fallback) {
      // ---- survivors, already in ascending id order (this overwrites sel and the member list)
      const uint32_t alive = hits | above;
      // one cursor walks through both staging arrays (the values sit kKcapMax words behind the ids): a
      // survivor is stored and moves the cursor on, everything else is predicated off
      static_assert(kKcapMax * 4 == 8192, "offset of st_vals behind st_ids in the store below");
      uint32_t at = smem_u32(sm.st_ids) + out_pos * 4u;
      auto stage_if = [&at](uint32_t id, float val, uint32_t bit) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %3, 0;\n\t@p st.shared.u32 [%0], %1;\n\t@p st.shared.f32 [%0+8192], %2;\n\t"
            "@p add.u32 %0, %0, 4;\n\t}"
            : "+r"(at)
            : "r"(id), "f"(val), "r"(bit)
            : "memory");
      };
#pragma unroll
      for (int j = 0; j < kPairChunk; ++j) {
        if ((uint32_t)j >= wcount) continue;
        const uint32_t id = 2u * ((j & 1) ? qq[j >> 1] >> 16 : qq[j >> 1] & 0xffffu);
        // a survivor is neither a NaN nor below tau0: adding zero is all that is left of canonical()
        stage_if(id, __fadd_rn(v[j].x, 0.0f), alive & (1u << (2 * j)));
        stage_if(id + 1u, __fadd_rn(v[j].y, 0.0f), alive & (2u << (2 * j)));
      }
    }
    group_sync<NT_P, BAR_P>();
    SJD_PHASE(20);
    if (fallback) {
      // redone by the any-shape path after the last row; the bins must be clear again for the next one
      for (int j = tid; j < kSelBins; j += NT_P) sm.sel[j] = 0;
      if (tid < kSelBins / 32) sm.sel_c[tid] = 0;
      if (tid == 0) sm.redo[sm.ctl[kRcRedo]++] = row;
      group_sync<NT_P, BAR_P>();
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
#pragma unroll
    for (int x = 0; x < kFinItems / 4; ++x) *reinterpret_cast<uint4*>(sm.sel + k0 + 4 * x) = make_uint4(0u, 0u, 0u, 0u);
    if (tid < kSelBins / 32) sm.sel_c[tid] = 0;
    const float Z = group_sum1_f32<NT_P, BAR_P>(zpart, tid, sm.scan_p, flip);
    SJD_PHASE(21);
    int32_t* out_ids = a.out_ids + (size_t)row * kcap;
    float* out_vals = a.out_vals + (size_t)row * kcap;
    uint64_t wgt[kFinItems], wloc = 0;
    float p[kFinItems];
    const float inv_Z = __fdiv_rn(1.0f, Z);  // one division per thread; p = e / Z within 1.5 ulp
#pragma unroll
    for (int j = 0; j < kFinItems; ++j) {
      p[j] = __fmul_rn(e[j], inv_Z);
      wgt[j] = fixed_weight(p[j]);
      wloc += wgt[j];
      if (ids[j] == draft && ids[j] >= 0) sm.ctl[kRcPtok] = __float_as_int(p[j]);
    }
    if ((kcap & 3) == 0 && k0 + kFinItems <= kcap) {
      int4* oi = reinterpret_cast<int4*>(out_ids + k0);
      float4* ov = reinterpret_cast<float4*>(out_vals + k0);
#pragma unroll
      for (int x = 0; x < kFinItems / 4; ++x) {
        oi[x] = make_int4(ids[4 * x], ids[4 * x + 1], ids[4 * x + 2], ids[4 * x + 3]);
        ov[x] = make_float4(p[4 * x], p[4 * x + 1], p[4 * x + 2], p[4 * x + 3]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < kFinItems; ++j) {
        if (k0 + j < kcap) {
          out_ids[k0 + j] = ids[j];
          out_vals[k0 + j] = p[j];
        }
      }
    }
    SJD_PHASE(22);
    // the row's own draw from p_i: fixed-point inverse CDF in ascending-id order
    uint64_t T;
    const uint64_t lo = group_scan1<NT_P, BAR_P, uint64_t>(wloc, tid, sm.scan_p, flip, &T);
    const uint64_t rnd64 = (uint64_t)(uint32_t)sm.ctl[kRcRndLo] | ((uint64_t)(uint32_t)sm.ctl[kRcRndHi] << 32);
    const uint64_t t = __umul64hi(rnd64, T);
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
    SJD_PHASE(23);
    SJD_PHASE_COUNT(40, 1);
    SJD_PHASE_COUNT(41, n_pairs);
  }
  // ---- rows the single pass could not finish: the exact any-shape path from global memory (rare).  Kept
  // out of the loop so that the loop holds no call and nothing of it lives across one.  Its scratch sits on
  // st_vals.
  group_sync<NT_P, BAR_P>();
  const int n_redo = dead ? 0 : sm.ctl[kRcRedo];
  for (int r = 0; r < n_redo; ++r)
    row_generic<DTYPE, NT_P, BAR_P>(a, sm.redo[r], tid, *reinterpret_cast<GenericSmem*>(sm.st_vals), kRowStatusRedone);
}

}  // namespace sjd

// Pipelined row kernel: the sampling head (guidance merge, temperature, top-K, softmax, per-row draw) in
// ONE pass over the logits, with the three parts of the work running concurrently on every SM.
//
// Persistent CTAs, one per SM, rows round-robin.  Three roles inside a CTA:
//
//   producer (1 warp)   streams each row through a ring of shared-memory stages with bulk asynchronous
//                       copies (cp.async.bulk, completion on mbarriers; no multicast, own CTA only).
//   filter (NF warps)   turns the staged bf16/fp32 pairs into merged logits y and keeps only the few per
//                       cent that can still be in the top-K.  The first stages of a row are a strided
//                       SAMPLE of it (every SS-th 256-element tile).  The maxima of the sample's groups
//                       of eight give a floor f below the sample's rank-m value; a linear histogram of
//                       the sample elements above f then gives the threshold tau0 whose rank in the sample
//                       is m, high enough that at least K elements of the row reach it (a row for which
//                       that fails is redone exactly, see below).  Pairs of neighbouring elements whose
//                       larger one reaches tau0 are appended to a per-thread list with branch-free
//                       arithmetic: the pair is always stored at the thread's cursor and the cursor
//                       advances only for a hit; one bit per pair records where the hits were.
//   finisher (NP warps) works on the PREVIOUS row while the filter streams the next one: turns lists
//                       and hit bits into a dense candidate list, finds the exact K-th largest
//                       (linear-bin histogram + ranking inside the threshold bin, ties to the lower
//                       id), orders the survivors by token id through a bitmap, and does softmax,
//                       coalesced output and the row's own inverse-CDF draw.
//
// A row whose candidates do not contain the top-K for sure (fewer than K of them) or do not fit the
// on-chip capacities is redone by row_generic() from global memory: the result is exact for any input.
//
// Every wait on an mbarrier is bounded (poll count and clock); on a time-out the CTA marks its
// remaining rows with kRowStatusTimeout, drains its own copies in flight and returns.
#pragma once

#include "device_utils.cuh"
#include "row_kernels.cuh"

namespace sjd {

constexpr int kTileElems = 256;           // elements per tile: one warp iteration, 8 per lane
constexpr int kStageArrayBytes = 8192;    // bytes of ONE logits array in a ring stage
constexpr int kHistBins = 2048;           // filter's sample histogram (group maxima by key, then linear bins)
constexpr int kSelBins = 2048;            // finisher's linear bins over [tau0, max]
constexpr int kListCap = 36;              // pair entries per filter thread and row (the last four are slack
                                          // for the unconditional stores of one tile)
constexpr int kMaskWordsMax = 8;          // 32 hit bits each: up to 64 tiles per filter warp and row
constexpr int kItersMax = 64;
constexpr int kDenseCap = 3072;           // candidates the finisher can hold for a row
constexpr int kBinListCap = 512;          // members of the threshold bin ranked by brute force
constexpr int kKcapMax = 2048;            // largest kcap the on-chip path stages
constexpr int kFinItems = 8;              // staged entries per finisher thread (kKcapMax / finisher threads)
constexpr uint32_t kSpinLimit = 1u << 22; // polls before a wait gives up
#ifdef SJD_TEST_SPIN_CYCLES
// test builds only: a short limit, so that a test can watch a wait run out (see SJD_TEST_DROP_COPY)
constexpr long long kSpinCycles = SJD_TEST_SPIN_CYCLES;
#else
constexpr long long kSpinCycles = 1ll << 31;  // ... or this many clock cycles, whichever comes first
#endif

struct PipeCfg {
  int sample_stride;  // SS: every SS-th tile of a row is a sample tile
  int sample_rank;    // m: rank (from the top) within the sample that fixes tau0
  int n_stages;       // ring depth
  int vwords;         // V / 32
  int mask_words;     // 32-bit words of hit bits per filter thread and row
};

struct Candidate {
  float y;
  int32_t id;
};

// ---------------------------------------------------------------------------------------------------
// PTX wrappers: mbarrier, 1-D bulk copy global -> shared, packed fp32 pairs
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the phase did not complete within kSpinLimit polls or kSpinCycles clocks.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && clock64() - t0 > kSpinCycles) break;
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// Two fp32 values in one 64-bit register; each half of a packed operation is rounded exactly like the
// scalar operation (round to nearest even, no flush to zero).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
// max of three; a NaN operand is ignored
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// ---------------------------------------------------------------------------------------------------
// Row schedule shared by the producer and the filter.
// Tiles of a row: g = 0 .. V/256-1.  Sample tiles: g % SS == 0.  The first `sample_stages` stages hold
// the sample tiles in order; the others hold the tail tiles t = 0.. in order, where tail tile t is
// global tile (t/(SS-1)) SS + 1 + t%(SS-1).
// ---------------------------------------------------------------------------------------------------
struct RowSchedule {
  int tiles, ss, sample_tiles, tail_tiles, sample_stages, stages;
  __device__ __forceinline__ RowSchedule(int V, int SS, int TPS) {
    ss = SS;
    tiles = V / kTileElems;
    sample_tiles = tiles / SS;
    tail_tiles = tiles - sample_tiles;
    sample_stages = (sample_tiles + TPS - 1) / TPS;
    stages = sample_stages + (tail_tiles + TPS - 1) / TPS;
  }
  __device__ __forceinline__ int stage_tiles(int s, int TPS) const {
    return s < sample_stages ? min(TPS, sample_tiles - TPS * s) : min(TPS, tail_tiles - TPS * (s - sample_stages));
  }
  __device__ __forceinline__ int global_tile(int s, int j, int TPS) const {
    if (s < sample_stages) return (s * TPS + j) * ss;
    const int t = TPS * (s - sample_stages) + j;
    const int run = t / (ss - 1);
    return run * ss + 1 + (t - run * (ss - 1));
  }
};

template <int DTYPE>
struct PipeTraits {
  static constexpr int kElemBytes = DTYPE == 0 ? 4 : 2;
  static constexpr int kTileBytes = kTileElems * kElemBytes;
  static constexpr int kTilesPerStage = kStageArrayBytes / kTileBytes;  // 16 (bf16) or 8 (fp32)
  static constexpr int kStageBytes = 2 * kStageArrayBytes;
};

// Element index inside a tile of the j-th value a lane holds.  bf16 / fp16: 8 consecutive elements per lane
// (one 16-byte load).  fp32: elements 4*lane..+3 and 128+4*lane..+3 (two conflict-free 16-byte loads).
template <int DTYPE>
__device__ __forceinline__ int tile_elem(int lane, int j) {
  if (DTYPE != 0) return lane * 8 + j;
  return j < 4 ? lane * 4 + j : 128 + lane * 4 + (j - 4);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// A thread's share of a staged tile as it lies in shared memory: 8 logits of each array.
template <int DTYPE>
struct RawTile {
  uint4 c[DTYPE != 0 ? 1 : 2];
  uint4 u[DTYPE != 0 ? 1 : 2];
};

template <int DTYPE, bool has_u>
__device__ __forceinline__ void load_raw(uint32_t ctile, uint32_t utile, int lane, RawTile<DTYPE>& r) {
  r.c[0] = lds128(ctile + lane * 16);
  if (DTYPE == 0) r.c[DTYPE != 0 ? 0 : 1] = lds128(ctile + 512 + lane * 16);
  if (has_u) {
    r.u[0] = lds128(utile + lane * 16);
    if (DTYPE == 0) r.u[DTYPE != 0 ? 0 : 1] = lds128(utile + 512 + lane * 16);
  }
}

// d = c - u for the two 16-bit values of word w, taken as they are (sm_100's subtract with one 16-bit operand
// widens it exactly): the same two roundings as widening by hand and subtracting, two instructions fewer.
template <int DTYPE>
__device__ __forceinline__ uint64_t sub2_narrow(uint32_t w, uint64_t u) {
  float u0, u1, d0, d1;
  unpack2(u, u0, u1);
  if (DTYPE == 1)
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tsub.rn.f32.bf16 %0, lo, %3;\n\tsub.rn.f32.bf16 %1, hi, %4;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "r"(w), "f"(u0), "f"(u1));
  else
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tsub.rn.f32.f16 %0, lo, %3;\n\tsub.rn.f32.f16 %1, hi, %4;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "r"(w), "f"(u0), "f"(u1));
  return pack2(d0, d1);
}

// Merged logits y of the thread's eight elements, as four packed pairs: d = c - u; g = fma(s, d, u);
// y = g * inv_T, one rounding per operation.  Multiplying by 1.0f is exact, so the last step is skipped
// when inv_T == 1.
template <int DTYPE, bool has_u, bool has_t>
__device__ __forceinline__ void merge_raw(const RawTile<DTYPE>& r, uint64_t s2, uint64_t t2, float (&y)[8]) {
  uint64_t c[4], u[4];
  if (DTYPE != 0 && has_u) {
    // guidance on 16-bit logits: only u is widened by hand, c goes into the subtraction as it is
    const uint4 w = r.c[0], v = r.u[0];
    const uint32_t cw[4] = {w.x, w.y, w.z, w.w}, uw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (DTYPE == 1) {
        u[k] = pack2(bf16_lo(uw[k]), bf16_hi(uw[k]));
      } else {
        const float2 uf = f16_pair(uw[k]);
        u[k] = pack2(uf.x, uf.y);
      }
      uint64_t g = fma2(s2, sub2_narrow<DTYPE>(cw[k], u[k]), u[k]);
      if (has_t) g = mul2(g, t2);
      unpack2(g, y[2 * k], y[2 * k + 1]);
    }
    return;
  }
  if (DTYPE == 1) {
    const uint4 w = r.c[0];
    c[0] = pack2(bf16_lo(w.x), bf16_hi(w.x)); c[1] = pack2(bf16_lo(w.y), bf16_hi(w.y));
    c[2] = pack2(bf16_lo(w.z), bf16_hi(w.z)); c[3] = pack2(bf16_lo(w.w), bf16_hi(w.w));
    if (has_u) {
      const uint4 v = r.u[0];
      u[0] = pack2(bf16_lo(v.x), bf16_hi(v.x)); u[1] = pack2(bf16_lo(v.y), bf16_hi(v.y));
      u[2] = pack2(bf16_lo(v.z), bf16_hi(v.z)); u[3] = pack2(bf16_lo(v.w), bf16_hi(v.w));
    }
  } else if (DTYPE == 2) {
    const uint4 w = r.c[0];
    const float2 c0 = f16_pair(w.x), c1 = f16_pair(w.y), c2 = f16_pair(w.z), c3 = f16_pair(w.w);
    c[0] = pack2(c0.x, c0.y); c[1] = pack2(c1.x, c1.y); c[2] = pack2(c2.x, c2.y); c[3] = pack2(c3.x, c3.y);
    if (has_u) {
      const uint4 v = r.u[0];
      const float2 u0 = f16_pair(v.x), u1 = f16_pair(v.y), u2 = f16_pair(v.z), u3 = f16_pair(v.w);
      u[0] = pack2(u0.x, u0.y); u[1] = pack2(u1.x, u1.y); u[2] = pack2(u2.x, u2.y); u[3] = pack2(u3.x, u3.y);
    }
  } else {
    const uint4 a = r.c[0], b = r.c[DTYPE != 0 ? 0 : 1];
    c[0] = (uint64_t)a.x | ((uint64_t)a.y << 32); c[1] = (uint64_t)a.z | ((uint64_t)a.w << 32);
    c[2] = (uint64_t)b.x | ((uint64_t)b.y << 32); c[3] = (uint64_t)b.z | ((uint64_t)b.w << 32);
    if (has_u) {
      const uint4 p = r.u[0], q = r.u[DTYPE != 0 ? 0 : 1];
      u[0] = (uint64_t)p.x | ((uint64_t)p.y << 32); u[1] = (uint64_t)p.z | ((uint64_t)p.w << 32);
      u[2] = (uint64_t)q.x | ((uint64_t)q.y << 32); u[3] = (uint64_t)q.z | ((uint64_t)q.w << 32);
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    uint64_t g = c[k];
    if (has_u) g = fma2(s2, sub2(c[k], u[k]), u[k]);
    if (has_t) g = mul2(g, t2);
    unpack2(g, y[2 * k], y[2 * k + 1]);
  }
}

template <int DTYPE, bool has_u, bool has_t>
__device__ __forceinline__ void tile_y8(uint32_t ctile, uint32_t utile, int lane, uint64_t s2, uint64_t t2,
                                        float (&y)[8]) {
  RawTile<DTYPE> r;
  load_raw<DTYPE, has_u>(ctile, utile, lane, r);
  merge_raw<DTYPE, has_u, has_t>(r, s2, t2, y);
}

// ---------------------------------------------------------------------------------------------------
// Shared-memory layout (dynamic)
// ---------------------------------------------------------------------------------------------------
enum {
  kCtlAbort = 0,  // a bounded wait gave up somewhere in this CTA
  // filter group
  kCtlFBin, kCtlFAbove, kCtlFCount, kCtlTau0, kCtlSmaxKey,
  // handed from the filter to the finisher with the row
  kCtlRowTau0, kCtlRowOverflow,
  // finisher group
  kCtlPBin, kCtlPAbove, kCtlPCount, kCtlGather, kCtlPtok, kCtlFoundId, kCtlFoundP,
  kCtlWords = 16
};

template <int NF>
struct PipeSmem {
  uint64_t* full;       // [n_stages]  ring: data landed
  uint64_t* empty;      // [n_stages]  ring: all filter warps done with the stage
  uint64_t* cand_full;  // lists and hit bits handed to the finisher
  uint64_t* cand_free;  // ... and handed back
  unsigned char* ring;  // [n_stages][2][kStageArrayBytes]
  uint64_t* ylist;      // [kListCap][NF*32]        pair entries, one column per filter thread
  uint32_t* masks;      // [mask_words][NF*32]      inverted hit bits, first pair in the top bit
  uint16_t* tile_of;    // [NF][kItersMax]          global tile of a filter warp's it-th tile of a row
  uint32_t* hist;       // [kHistBins]     (filter)
  Candidate* dense;     // [kDenseCap]     (finisher)
  int32_t* st_ids;      // [kKcapMax]      (finisher) staging, ascending id
  float* st_vals;       // [kKcapMax]
  uint32_t* sel;        // [kSelBins]      (finisher) = st_ids: dead before the staging is written
  Candidate* binlist;   // [kBinListCap]   (finisher) = st_vals: likewise
  uint32_t* bitmap;     // [vwords]        (finisher)
  uint16_t* wprefix;    // [vwords]        (finisher)
  uint64_t* scan_f;     // group scratch, filter
  uint64_t* scan_p;     // group scratch, finisher
  int* ctl;             // control words
};

__host__ __device__ inline size_t pipe_smem_fixed_bytes(int NF, int vwords, int mask_words) {
  size_t b = 0;
  b += 32 * 8;                                           // mbarriers (2 per ring stage + 2)
  b += (size_t)kListCap * NF * 32 * 8;                   // ylist
  b += (size_t)mask_words * NF * 32 * 4;                 // masks
  b += (size_t)NF * kItersMax * 2;                       // tile_of
  b += (size_t)kHistBins * 4;
  b += (size_t)kDenseCap * sizeof(Candidate);
  b += (size_t)kKcapMax * 8;
  b += (size_t)vwords * 4 + (size_t)vwords * 2;
  b += 2 * (2 * 32 + 8) * 8;
  b += kCtlWords * 4;
  return b + 128;  // alignment slack
}
__host__ __device__ inline size_t pipe_smem_bytes(int n_stages, int NF, int vwords, int mask_words) {
  return pipe_smem_fixed_bytes(NF, vwords, mask_words) + (size_t)n_stages * 2 * kStageArrayBytes;
}

template <int NF>
__device__ __forceinline__ PipeSmem<NF> carve_pipe_smem(unsigned char* base, int n_stages, int vwords, int mask_words) {
  static_assert(sizeof(uint32_t) * kSelBins <= sizeof(int32_t) * kKcapMax, "sel must fit under st_ids");
  static_assert(sizeof(Candidate) * kBinListCap <= sizeof(float) * kKcapMax, "binlist must fit under st_vals");
  PipeSmem<NF> s;
  // plain pointer arithmetic on the shared array, so that the compiler keeps the shared address space
  unsigned char* p = base + ((128u - (smem_u32(base) & 127u)) & 127u);
  s.ring = p;
  p += (size_t)n_stages * 2 * kStageArrayBytes;
  s.ylist = reinterpret_cast<uint64_t*>(p);
  p += (size_t)kListCap * NF * 32 * 8;
  s.dense = reinterpret_cast<Candidate*>(p);
  p += (size_t)kDenseCap * sizeof(Candidate);
  s.st_ids = reinterpret_cast<int32_t*>(p);
  s.sel = reinterpret_cast<uint32_t*>(p);
  p += (size_t)kKcapMax * 4;
  s.st_vals = reinterpret_cast<float*>(p);
  s.binlist = reinterpret_cast<Candidate*>(p);
  p += (size_t)kKcapMax * 4;
  s.hist = reinterpret_cast<uint32_t*>(p);
  p += (size_t)kHistBins * 4;
  s.masks = reinterpret_cast<uint32_t*>(p);
  p += (size_t)mask_words * NF * 32 * 4;
  s.bitmap = reinterpret_cast<uint32_t*>(p);
  p += (size_t)vwords * 4;
  s.full = reinterpret_cast<uint64_t*>(p);
  s.empty = s.full + n_stages;
  s.cand_full = s.empty + n_stages;
  s.cand_free = s.cand_full + 1;
  p += 32 * 8;
  s.scan_f = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.scan_p = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.ctl = reinterpret_cast<int*>(p);
  p += kCtlWords * 4;
  s.tile_of = reinterpret_cast<uint16_t*>(p);
  p += (size_t)NF * kItersMax * 2;
  s.wprefix = reinterpret_cast<uint16_t*>(p);
  return s;
}

// Largest bin b with (entries in bins > b) < target <= (entries in bins >= b).  The count above it goes
// to ctl[c_bin + 1], the bin's own count to ctl[c_bin + 2]; ctl[c_bin] = -1 when the histogram holds
// fewer than `target` entries.  All NT threads of the group call it; every bin is read by exactly one
// thread, which leaves it zero for its next use.  Two barriers.
template <int BINS, int NT, int BAR>
__device__ __forceinline__ void find_rank_bin(uint32_t* hist, uint32_t target, int tid, uint64_t* scratch, int& flip,
                                              int* ctl, int c_bin) {
  constexpr int PER = BINS / NT;
  static_assert(BINS % NT == 0 && PER % 4 == 0, "bins must split into 16-byte pieces per thread");
  // thread t owns bins BINS-1 - PER*t - j, j = 0..PER-1, i.e. words [BINS - PER (t+1), BINS - PER t)
  uint32_t c[PER], sum = 0;
  uint4* mine = reinterpret_cast<uint4*>(hist + BINS - PER * (tid + 1));
#pragma unroll
  for (int v = 0; v < PER / 4; ++v) {
    const uint4 w = mine[v];
    mine[v] = make_uint4(0u, 0u, 0u, 0u);
    c[PER - 1 - 4 * v] = w.x; c[PER - 2 - 4 * v] = w.y; c[PER - 3 - 4 * v] = w.z; c[PER - 4 - 4 * v] = w.w;
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) sum += c[j];
  if (tid == 0) ctl[c_bin] = -1;  // ordered before the owner's write by the barrier inside the scan
  uint32_t total;
  uint32_t above = group_scan1<NT, BAR, uint32_t>(sum, tid, scratch, flip, &total);
  if (above < target && target <= above + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (above < target && target <= above + c[j]) {
        ctl[c_bin] = BINS - 1 - PER * tid - j;
        ctl[c_bin + 1] = (int)above;
        ctl[c_bin + 2] = (int)c[j];
      }
      above += c[j];
    }
  }
  group_sync<NT, BAR>();
}

// float of an order-preserving key (inverse of float_key)
__device__ __forceinline__ float key_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// The filter warps' loop over this CTA's rows (see the head of the file).  BAR_F = 1 is their named barrier.
template <int DTYPE, int NF, bool HAS_U, bool HAS_T>
__device__ __forceinline__ void filter_role(const RowArgs& a, const PipeCfg& cfg, const PipeSmem<NF>& sm,
                                            const RowSchedule& sched) {
  constexpr int NT_F = NF * 32;
  constexpr int BAR_F = 1;
  constexpr uint32_t kStride = NT_F * 8;  // bytes between consecutive entries of one filter thread
  using TR = PipeTraits<DTYPE>;
  constexpr int TPS = TR::kTilesPerStage;
  const int tid = threadIdx.x, lane = threadIdx.x & 31, fw = threadIdx.x >> 5;
  const int NS = cfg.n_stages, mask_words = cfg.mask_words;
  const int rows = a.B * a.W;
  const float neg_inf = __int_as_float(0xff800000);
  const float lowest = -3.402823466e38f;  // with this threshold every finite value is a candidate
  volatile int* abort_flag = sm.ctl + kCtlAbort;
  const uint64_t s2 = pack2(a.s, a.s), t2 = pack2(a.inv_T, a.inv_T);
  const uint32_t ring_addr = smem_u32(sm.ring);
  const uint32_t list_base = smem_u32(sm.ylist) + (uint32_t)tid * 8u;
  const uint32_t list_limit = list_base + (uint32_t)(kListCap - 4) * kStride;  // beyond it a tile may not fit
  int slot = 0, flip = 0;
  uint32_t phase = 0;
  uint32_t n_row = 0;
  bool dead = false;
  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    // from the block's last row on, the verification grid may be scheduled (it waits for this grid's end)
    if (row + (int)gridDim.x >= rows) allow_dependent_launch();
    const int b = row / a.W, i = row - b * a.W;
    const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
    if (i >= L || dead) continue;

    // ---------------- sample, first pass: maxima of groups of eight, by key ----------------
    bool ok = true;
    float smax = neg_inf;
    {
      int sl = slot;
      uint32_t ph = phase;
      for (int s = 0; s < sched.sample_stages && ok; ++s) {
        ok = mbar_wait(&sm.full[sl], ph);
        if (ok) {
          const uint32_t st_c = ring_addr + (uint32_t)sl * TR::kStageBytes;
          const uint32_t st_u = st_c + kStageArrayBytes;
          const int nt = sched.stage_tiles(s, TPS);
          for (int j = fw; j < nt; j += NF) {
            float y[8];
            tile_y8<DTYPE, HAS_U, HAS_T>(st_c + (uint32_t)j * TR::kTileBytes, st_u + (uint32_t)j * TR::kTileBytes, lane, s2,
                                         t2, y);
            const float m8 = max3(max3(max3(neg_inf, y[0], y[1]), y[2], y[3]), max3(y[4], y[5], y[6]), y[7]);
            atomicAdd(&sm.hist[float_key(canonical(m8)) >> 21], 1u);
            smax = fmaxf(smax, m8);
          }
        }
        if (++sl == NS) {
          sl = 0;
          ph ^= 1u;
        }
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, d));
    if (lane == 0) atomicMax(reinterpret_cast<unsigned int*>(&sm.ctl[kCtlSmaxKey]), float_key(canonical(smax)));
    // lists and hit bits must be back from the finisher before anything is appended
    if (ok && n_row > 0) ok = mbar_wait(sm.cand_free, (n_row - 1) & 1u);
    dead = group_any<NT_F, BAR_F>(!ok);
    if (dead) {
      if (tid == 0) *abort_flag = 1;
      continue;
    }
    // at least m group maxima, hence at least m sample elements, are >= the lower edge of this bin
    find_rank_bin<kHistBins, NT_F, BAR_F>(sm.hist, (uint32_t)cfg.sample_rank, tid, sm.scan_f, flip, sm.ctl, kCtlFBin);
    const int cbin = sm.ctl[kCtlFBin];
    float floor_y = cbin >= 0 ? key_float((uint32_t)cbin << 21) : lowest;
    if (!(floor_y >= lowest)) floor_y = lowest;  // edge fell on -inf or into the NaN patterns
    const float top_y = key_float((uint32_t)sm.ctl[kCtlSmaxKey]);
    const bool refine = floor_y > lowest && top_y >= floor_y && top_y <= 3.402823466e38f;
    const float range = __fsub_rn(top_y, floor_y);
    const float scale = (refine && range > 0.0f) ? __fdiv_rn((float)kHistBins - 0.5f, range) : 0.0f;

    uint32_t cur = list_base;  // shared-memory address of the thread's next free entry
    uint32_t imw = 0;          // inverted hit bits of the last (it & 7) tiles
    int it = 0;                // tiles this warp has filtered in this row
    bool overflow = false;
    // One tile: four pairs.  A pair is always stored at the cursor; the cursor moves on only for a hit,
    // i.e. when max(pair) >= thr.  A pair of NaNs and -inf never hit.
    auto filter_tile = [&](uint32_t ctile, uint32_t utile, float thr) {
      float y[8];
      tile_y8<DTYPE, HAS_U, HAS_T>(ctile, utile, lane, s2, t2, y);
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
      ++it;
      if ((it & 7) == 0) {
        if ((it >> 3) <= mask_words) sm.masks[(size_t)((it >> 3) - 1) * NT_F + tid] = imw;
        imw = 0;
      }
    };
    // ---------------- the sample tiles against the floor (a superset of what tau0 will keep) ----------------
    const float sample_thr = refine ? floor_y : lowest;
    for (int s = 0; s < sched.sample_stages; ++s) {
      const uint32_t st_c = ring_addr + (uint32_t)slot * TR::kStageBytes;
      const uint32_t st_u = st_c + kStageArrayBytes;
      const int nt = sched.stage_tiles(s, TPS);
      for (int j = fw; j < nt; j += NF)
        filter_tile(st_c + (uint32_t)j * TR::kTileBytes, st_u + (uint32_t)j * TR::kTileBytes, sample_thr);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[slot]);
      if (++slot == NS) {
        slot = 0;
        phase ^= 1u;
      }
    }
    // ---------------- sample, second pass: linear bins over [floor, sample max], from the lists ----------------
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
      if (tid == 0) sm.ctl[kCtlSmaxKey] = 0;  // every thread has read it; next written after the next row's barriers
      find_rank_bin<kHistBins, NT_F, BAR_F>(sm.hist, (uint32_t)cfg.sample_rank, tid, sm.scan_f, flip, sm.ctl, kCtlFBin);
      const int fbin = sm.ctl[kCtlFBin];
      if (fbin > 0 && scale > 0.0f) {
        // a little below the lower edge of the bin, so that rounding cannot exclude one of its members
        const float t = __fmul_rd(__fdiv_rd((float)fbin, scale), 0.99999f);
        tau0 = __fadd_rd(floor_y, t);
      } else if (fbin >= 0) {
        tau0 = floor_y;
      }
    } else {
      group_sync<NT_F, BAR_F>();
      if (tid == 0) sm.ctl[kCtlSmaxKey] = 0;
    }
    // ---------------- the rest of the row against tau0 ----------------
    for (int s = sched.sample_stages; s < sched.stages; ++s) {
      if (ok) ok = mbar_wait(&sm.full[slot], phase);
      if (ok) {
        const uint32_t st_c = ring_addr + (uint32_t)slot * TR::kStageBytes;
        const uint32_t st_u = st_c + kStageArrayBytes;
        const int nt = sched.stage_tiles(s, TPS);
        for (int j = fw; j < nt; j += NF)
          filter_tile(st_c + (uint32_t)j * TR::kTileBytes, st_u + (uint32_t)j * TR::kTileBytes, tau0);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[slot]);
      if (++slot == NS) {
        slot = 0;
        phase ^= 1u;
      }
    }
    // ---------------- hand the row over ----------------
    {
      const int rem = it & 7;
      int w = it >> 3;
      if (rem != 0 && w < mask_words) {
        const int fill = 32 - 4 * rem;  // bits of the word not reached: misses
        sm.masks[(size_t)w * NT_F + tid] = (imw << fill) | ((1u << fill) - 1u);
        ++w;
      }
      for (; w < mask_words; ++w) sm.masks[(size_t)w * NT_F + tid] = 0xffffffffu;
      if (overflow) sm.ctl[kCtlRowOverflow] = 1;
      if (tid == 0) sm.ctl[kCtlRowTau0] = __float_as_int(tau0);
    }
    dead = group_any<NT_F, BAR_F>(!ok);
    if (dead) {
      if (tid == 0) *abort_flag = 1;
      continue;  // the row is not handed over: the finisher's wait runs out and marks the rows
    }
    if (lane == 0) mbar_arrive(sm.cand_full);
    ++n_row;
  }
}

template <int DTYPE, int NF, int NP>
__global__ void __launch_bounds__((NF + NP + 1) * 32, 1) rows_pipeline_kernel(const RowArgs a, const PipeCfg cfg) {
  constexpr int NT_F = NF * 32, NT_P = NP * 32;
  constexpr int BAR_P = 2;  // named barrier of the finisher warps (the filter warps use 1)
  static_assert(NF <= 16 && NP * 32 * kFinItems >= kKcapMax, "group sizes");
  using TR = PipeTraits<DTYPE>;
  constexpr int TPS = TR::kTilesPerStage;
  extern __shared__ unsigned char smem_raw[];
  PipeSmem<NF> sm = carve_pipe_smem<NF>(smem_raw, cfg.n_stages, cfg.vwords, cfg.mask_words);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NS = cfg.n_stages;
  const bool has_u = a.uncond != nullptr;
  const float neg_inf = __int_as_float(0xff800000);

  const RowSchedule sched(a.V, cfg.sample_stride, TPS);
  const int rows = a.B * a.W;
  const int mask_words = cfg.mask_words;

  // ---- one-time set-up: barriers, the tables that must start at zero, the tile map ----
  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], NF);
    }
    mbar_init(sm.cand_full, NF);
    mbar_init(sm.cand_free, 1);
    for (int k = 0; k < kCtlWords; ++k) sm.ctl[k] = 0;
    fence_barrier_init();
  }
  for (int j = threadIdx.x; j < kHistBins; j += blockDim.x) sm.hist[j] = 0;
  for (int j = threadIdx.x; j < kSelBins; j += blockDim.x) sm.sel[j] = 0;
  for (int j = threadIdx.x; j < cfg.vwords; j += blockDim.x) sm.bitmap[j] = 0;
  if (warp < NF && lane == 0) {
    int it = 0;
    for (int s = 0; s < sched.stages; ++s) {
      const int nt = sched.stage_tiles(s, TPS);
      for (int j = warp; j < nt; j += NF)
        if (it < kItersMax) sm.tile_of[warp * kItersMax + it++] = (uint16_t)sched.global_tile(s, j, TPS);
    }
  }
  // only shared memory so far; a launch allowed to overlap the stream's previous kernel waits for its end here
  grid_dependency_wait();
  __syncthreads();

  volatile int* abort_flag = sm.ctl + kCtlAbort;

  if (warp == NF + NP) {
    // ====================================== producer warp ======================================
    int slot = 0;
    uint32_t use = 0;   // how many times `slot` has been filled before
    uint32_t issued = 0;
    bool ok = true;
    for (int row = blockIdx.x; row < rows && ok; row += gridDim.x) {
      const int b = row / a.W, i = row - b * a.W;
      const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
      if (i >= L) continue;
      const int64_t off = (int64_t)b * a.stride_b + (int64_t)i * a.stride_w;
      const unsigned char* gc = static_cast<const unsigned char*>(a.cond) + off * TR::kElemBytes;
      const unsigned char* gu = has_u ? static_cast<const unsigned char*>(a.uncond) + off * TR::kElemBytes : nullptr;
      for (int s = 0; s < sched.stages; ++s) {
        if (use > 0) ok = mbar_wait(&sm.empty[slot], (use - 1) & 1u);
        ok = __all_sync(0xffffffffu, ok && (*abort_flag == 0));
        if (!ok) break;
        const int nt = sched.stage_tiles(s, TPS);
        unsigned char* dst_c = sm.ring + (size_t)slot * TR::kStageBytes;
        unsigned char* dst_u = dst_c + kStageArrayBytes;
        if (lane == 0) mbar_arrive_expect_tx(&sm.full[slot], (uint32_t)nt * TR::kTileBytes * (has_u ? 2u : 1u));
        __syncwarp();
        if (s < sched.sample_stages) {
          // sample tiles are isolated in the row: one copy per tile, spread over the lanes
          for (int j = lane; j < nt; j += 32) {
            const size_t goff = (size_t)(s * TPS + j) * sched.ss * TR::kTileBytes;
            bulk_g2s(dst_c + (uint32_t)j * TR::kTileBytes, gc + goff, TR::kTileBytes, &sm.full[slot]);
            if (has_u) bulk_g2s(dst_u + (uint32_t)j * TR::kTileBytes, gu + goff, TR::kTileBytes, &sm.full[slot]);
          }
        } else {
          // tail tiles come in runs of SS-1 contiguous tiles: lane r copies the r-th run of the stage
          const int t0 = TPS * (s - sched.sample_stages), t1 = t0 + nt, rl = sched.ss - 1;
          const int run = t0 / rl + lane;
          const int ta = max(run * rl, t0), tb = min((run + 1) * rl, t1);
          if (ta < tb) {
            const int g = run * sched.ss + 1 + (ta - run * rl);
            const uint32_t bytes = (uint32_t)(tb - ta) * TR::kTileBytes;
            const size_t goff = (size_t)g * TR::kTileBytes, soff = (size_t)(ta - t0) * TR::kTileBytes;
            bulk_g2s(dst_c + soff, gc + goff, bytes, &sm.full[slot]);
            if (has_u) bulk_g2s(dst_u + soff, gu + goff, bytes, &sm.full[slot]);
          }
        }
        ++issued;
        if (++slot == NS) {
          slot = 0;
          ++use;
        }
      }
    }
    // drain: every stage this warp armed must have landed before the CTA may exit
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
      if (!ok && lane == 0) *abort_flag = 1;
    }
    return;
  }

  if (warp < NF) {
    // ======================================= filter warps =======================================
    const bool has_t = a.inv_T != 1.0f;
    if (has_u) {
      if (has_t) filter_role<DTYPE, NF, true, true>(a, cfg, sm, sched);
      else filter_role<DTYPE, NF, true, false>(a, cfg, sm, sched);
    } else {
      if (has_t) filter_role<DTYPE, NF, false, true>(a, cfg, sm, sched);
      else filter_role<DTYPE, NF, false, false>(a, cfg, sm, sched);
    }
    return;
  }

  // ======================================= finisher warps =======================================
  const int tid = threadIdx.x - NT_F;  // 0 .. NT_P-1
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
    const float tau0 = __int_as_float(sm.ctl[kCtlRowTau0]);
    bool fallback = kcap > kKcapMax || sm.ctl[kCtlRowOverflow] != 0;

    // ---- lists + hit bits -> dense candidate list.  Pass 1 counts the values that reach tau0 ----
    uint32_t my_valid = 0;
    if (!fallback) {
      for (int col = tid; col < NT_F; col += NT_P) {
        int n_e = 0;
        for (int w = 0; w < mask_words; ++w) n_e += __popc(~sm.masks[(size_t)w * NT_F + col]);
        n_e = min(n_e, kListCap);
        for (int e = 0; e < n_e; ++e) {
          const float2 pr = *reinterpret_cast<const float2*>(&sm.ylist[(size_t)e * NT_F + col]);
          my_valid += (pr.x >= tau0 ? 1u : 0u) + (pr.y >= tau0 ? 1u : 0u);
        }
      }
    }
    uint32_t n_total;
    uint32_t my_off = group_scan1<NT_P, BAR_P, uint32_t>(my_valid, tid, sm.scan_p, flip, &n_total);
    fallback |= n_total < (uint32_t)kcap || n_total > (uint32_t)kDenseCap;
    // ---- pass 2 decodes the token ids from the hit bits and writes the dense list ----
    float vmax = neg_inf;
    if (!fallback) {
      for (int col = tid; col < NT_F; col += NT_P) {
        const int cw = col >> 5, cl = col & 31;
        int e = 0;
        for (int w = 0; w < mask_words; ++w) {
          uint32_t x = ~sm.masks[(size_t)w * NT_F + col];
          while (x != 0u && e < kListCap) {
            const int bitpos = __clz((int)x);
            x &= ~(0x80000000u >> bitpos);
            const int q = w * 32 + bitpos;  // pair index within the row for this thread
            const int tile = sm.tile_of[cw * kItersMax + (q >> 2)];
            const int id = tile * kTileElems + tile_elem<DTYPE>(cl, 2 * (q & 3));
            const float2 pr = *reinterpret_cast<const float2*>(&sm.ylist[(size_t)e * NT_F + col]);
            ++e;
            if (pr.x >= tau0) {
              sm.dense[my_off++] = Candidate{pr.x, id};
              vmax = fmaxf(vmax, pr.x);
            }
            if (pr.y >= tau0) {
              sm.dense[my_off++] = Candidate{pr.y, id + 1};
              vmax = fmaxf(vmax, pr.y);
            }
          }
        }
      }
    }
    vmax = group_max1_f32<NT_P, BAR_P>(vmax, tid, sm.scan_p, flip);
    // lists and hit bits are not read again: hand them back
    if (tid == 0) {
      sm.ctl[kCtlRowOverflow] = 0;
      sm.ctl[kCtlGather] = 0;
      sm.ctl[kCtlPtok] = 0;
      sm.ctl[kCtlFoundId] = -1;
      mbar_arrive(sm.cand_free);
    }
    ++n_row;
    fallback |= !(vmax <= 3.402823466e38f);  // an infinite logit: the any-shape path decides what the row is

    // visit the dense list, four independent entries per thread in flight
    auto for_each_candidate = [&](auto f) {
      for (uint32_t i0 = 0; i0 < n_total; i0 += 4 * NT_P) {
        Candidate c[4];
        bool v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t ix = i0 + q * NT_P + tid;
          v[q] = ix < n_total;
          if (v[q]) c[q] = sm.dense[ix];
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (v[q]) f(c[q]);
      }
    };
    int tbin = 0, need = 0, nbin = 0;
    const float range = __fsub_rn(vmax, tau0);
    const float scale = range > 0.0f ? __fdiv_rn((float)kSelBins * 0.999f, range) : 0.0f;
    // linear bins over [tau0, vmax]; monotone in y, so a higher bin holds strictly larger values
    auto bin_of = [&](float y) {
      const int q = __float2int_rd(__fmul_rn(__fsub_rn(y, tau0), scale));
      return min(max(q, 0), kSelBins - 1);
    };
    if (!fallback) {
      for_each_candidate([&](const Candidate& c) { atomicAdd(&sm.sel[bin_of(c.y)], 1u); });
      group_sync<NT_P, BAR_P>();
      find_rank_bin<kSelBins, NT_P, BAR_P>(sm.sel, (uint32_t)kcap, tid, sm.scan_p, flip, sm.ctl, kCtlPBin);
      tbin = sm.ctl[kCtlPBin];
      need = kcap - sm.ctl[kCtlPAbove];  // members of the threshold bin that survive
      nbin = sm.ctl[kCtlPCount];
      if (tbin < 0 || nbin > kBinListCap) fallback = true;
    }
    const int wper = (cfg.vwords + NT_P - 1) / NT_P;
    const int w0 = min(tid * wper, cfg.vwords), w1 = min(w0 + wper, cfg.vwords);
    if (!fallback) {
      // ---- survivors into the bitmap over token ids: everything above the threshold bin, and the
      //      `need` best of the bin itself by (y descending, id ascending) ----
      for_each_candidate([&](const Candidate& c) {
        const int q = bin_of(c.y);
        if (q > tbin) atomicOr(&sm.bitmap[c.id >> 5], 1u << (c.id & 31));
        else if (q == tbin) sm.binlist[atomicAdd(&sm.ctl[kCtlGather], 1)] = Candidate{canonical(c.y), c.id};
      });
      group_sync<NT_P, BAR_P>();
      for (int x = tid; x < nbin; x += NT_P) {
        const Candidate me = sm.binlist[x];
        int rank = 0;
        for (int z = 0; z < nbin; ++z) {
          const Candidate o = sm.binlist[z];
          rank += (o.y > me.y || (o.y == me.y && o.id < me.id)) ? 1 : 0;
        }
        if (rank < need) atomicOr(&sm.bitmap[me.id >> 5], 1u << (me.id & 31));
      }
      group_sync<NT_P, BAR_P>();
      // ---- exclusive prefix of the per-word popcounts; each thread owns a contiguous run of words ----
      uint32_t wsum = 0;
      for (int w = w0; w < w1; ++w) wsum += __popc(sm.bitmap[w]);
      uint32_t total;
      uint32_t wrun = group_scan1<NT_P, BAR_P, uint32_t>(wsum, tid, sm.scan_p, flip, &total);
      for (int w = w0; w < w1; ++w) {
        sm.wprefix[w] = (uint16_t)wrun;
        wrun += __popc(sm.bitmap[w]);
      }
      if (total != (uint32_t)kcap) fallback = true;  // cannot happen; keep the result exact anyway
      group_sync<NT_P, BAR_P>();
    }
    if (!fallback) {
      // ---- softmax numerators into ascending-id order (this overwrites sel and binlist) ----
      for_each_candidate([&](const Candidate& c) {
        const uint32_t w = sm.bitmap[c.id >> 5];
        const uint32_t bit = 1u << (c.id & 31);
        if (w & bit) {
          const int p = (int)sm.wprefix[c.id >> 5] + __popc(w & (bit - 1u));
          sm.st_ids[p] = c.id;
          sm.st_vals[p] = exp_diff(canonical(c.y), vmax);
        }
      });
    }
    group_sync<NT_P, BAR_P>();
    for (int w = w0; w < w1; ++w) sm.bitmap[w] = 0;
    if (fallback) {
      // exact any-shape path from global memory (the row is still in L2); its scratch sits on st_vals,
      // so that sel (= st_ids) stays zero
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
      e[j] = in ? sm.st_vals[k0 + j] : 0.0f;
      ids[j] = in ? sm.st_ids[k0 + j] : -1;
      zpart += e[j];
    }
    // these eight words of st_ids are this thread's share of sel: zero again for the next row
    if (k0 + kFinItems <= kSelBins) {
      *reinterpret_cast<uint4*>(sm.sel + k0) = make_uint4(0u, 0u, 0u, 0u);
      *reinterpret_cast<uint4*>(sm.sel + k0 + 4) = make_uint4(0u, 0u, 0u, 0u);
    }
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
      if (ids[j] == draft && ids[j] >= 0) sm.ctl[kCtlPtok] = __float_as_int(p[j]);
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
      sm.ctl[kCtlFoundId] = fid;
      sm.ctl[kCtlFoundP] = __float_as_int(fp);
    }
    if (T == 0 && tid == 0) {  // all weights rounded to zero: take the first entry
      sm.ctl[kCtlFoundId] = ids[0];
      sm.ctl[kCtlFoundP] = __float_as_int(p[0]);
    }
    group_sync<NT_P, BAR_P>();
    if (tid == 0) {
      a.out_cnt[row] = kcap;
      *rs = RowScratch{__int_as_float(sm.ctl[kCtlPtok]), sm.ctl[kCtlFoundId], __int_as_float(sm.ctl[kCtlFoundP]), 0};
    }
    group_sync<NT_P, BAR_P>();
  }
}

}  // namespace sjd

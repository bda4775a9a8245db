// Streaming row kernel: the sampling head (guidance merge, temperature, top-K, softmax, per-row draw) in
// ONE pass over the logits.
//
// Persistent CTAs, one per SM.  A producer warp streams each row through a ring of shared-memory stages
// with bulk asynchronous copies (cp.async.bulk, completion on mbarriers); consumer warps turn the staged
// bf16/fp32 pairs into merged logits y and keep only the few per cent that can still be in the top-K:
//
//   1. The first stage of a row is a strided SAMPLE of it (every SS-th 256-element tile).  A 4096-bin
//      histogram of the sample's order-preserving keys gives a threshold tau0 whose rank in the sample
//      is high enough that, with overwhelming probability, at least K elements of the row reach it.
//   2. Every element with y >= tau0 (sample stage included) is appended to a per-thread candidate list
//      in shared memory; nothing else of the row is kept.
//   3. The exact K-th largest candidate (ties to the lower id) is found by one linear-bin histogram
//      plus a brute-force ranking inside the threshold bin; a bitmap over token ids gives each survivor
//      its position in ascending-id order; softmax, output and the row's own draw follow.
//
// A row whose candidates do not contain the top-K for sure (fewer than K of them), or do not fit the
// on-chip capacities, is redone by row_generic() from global memory: the result is always exact.
//
// Every wait on an mbarrier is bounded; on a time-out the CTA marks its remaining rows with
// kRowStatusTimeout, drains its own copies in flight and returns.
#pragma once

#include "device_utils.cuh"
#include "row_kernels.cuh"

namespace sjd {

constexpr int kTileElems = 256;           // elements per tile: one warp iteration, 8 per lane
constexpr int kStageBytesPerArray = 16384;
constexpr int kHistBins = 4096;
constexpr int kLaneListCap = 16;          // candidate entries owned by one consumer thread
constexpr int kOverflowCap = 1024;        // shared spill list
constexpr int kBinListCap = 1024;         // members of the threshold bin ranked by brute force
constexpr int kStageKcapMax = 2048;       // largest kcap the on-chip path stages
constexpr uint32_t kSpinLimit = 1u << 22; // polls before a wait gives up

struct StreamCfg {
  int sample_stride;  // SS: every SS-th tile of a row is a sample tile
  int sample_rank;    // m: rank (from the top) within the sample that fixes tau0
  int n_stages;       // ring depth
  int vwords;         // V / 32
};

struct Candidate {
  float y;
  int32_t id;
};

// ---------------------------------------------------------------------------------------------------
// PTX wrappers: mbarrier and 1-D bulk copy global -> shared (no multicast, own CTA only)
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// Bounded wait: false when the barrier did not flip within kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------------
// Row schedule shared by the producer and the consumers.
// Tiles of a row: g = 0 .. V/256-1.  Sample tiles: g % SS == 0.  Stage 0 holds the sample tiles, stage
// s >= 1 holds tail tiles t in [TPS (s-1), TPS s), where tail tile t is global tile (t/(SS-1)) SS + 1 + t%(SS-1).
// ---------------------------------------------------------------------------------------------------
struct RowSchedule {
  int tiles, sample_tiles, tail_tiles, stages, ss;
  __device__ __forceinline__ RowSchedule(int V, int SS, int TPS) {
    ss = SS;
    tiles = V / kTileElems;
    sample_tiles = tiles / SS;
    tail_tiles = tiles - sample_tiles;
    stages = 1 + (tail_tiles + TPS - 1) / TPS;
  }
  __device__ __forceinline__ int stage_tiles(int s, int TPS) const {
    return s == 0 ? sample_tiles : min(TPS, tail_tiles - TPS * (s - 1));
  }
  __device__ __forceinline__ int global_tile(int s, int j, int TPS) const {
    if (s == 0) return j * ss;
    const int t = TPS * (s - 1) + j;
    const int run = t / (ss - 1);
    return run * ss + 1 + (t - run * (ss - 1));
  }
};

template <int DTYPE>
struct StreamTraits {
  static constexpr int kElemBytes = DTYPE == 1 ? 2 : 4;
  static constexpr int kTileBytes = kTileElems * kElemBytes;
  static constexpr int kTilesPerStage = kStageBytesPerArray / kTileBytes;  // 32 (bf16) or 16 (fp32)
  static constexpr int kStageBytes = 2 * kStageBytesPerArray;
};

// Eight logits of one lane from a staged tile.  bf16: elements 8*lane..8*lane+7 (one 16-byte load).
// fp32: elements 4*lane..+3 and 128+4*lane..+3 (two conflict-free 16-byte loads).
template <int DTYPE>
__device__ __forceinline__ void tile_load8(const unsigned char* tile, int lane, float (&x)[8]) {
  if (DTYPE == 1) {
    const uint4 w = *reinterpret_cast<const uint4*>(tile + lane * 16);
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
  } else {
    const float4 a = *reinterpret_cast<const float4*>(tile + lane * 16);
    const float4 b = *reinterpret_cast<const float4*>(tile + 512 + lane * 16);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  }
}
template <int DTYPE>
__device__ __forceinline__ int tile_elem(int lane, int j) {
  if (DTYPE == 1) return lane * 8 + j;
  return j < 4 ? lane * 4 + j : 128 + lane * 4 + (j - 4);
}

// Merged logits of the lane's eight elements of a staged tile.  NaN compares false against any
// threshold and therefore never becomes a candidate, which is how a masked entry behaves.
template <int DTYPE>
__device__ __forceinline__ void tile_y8(const unsigned char* ctile, const unsigned char* utile, bool has_u, int lane,
                                        float s, float inv_T, float (&y)[8]) {
  float c[8];
  tile_load8<DTYPE>(ctile, lane, c);
  if (has_u) {
    float u[8];
    tile_load8<DTYPE>(utile, lane, u);
#pragma unroll
    for (int j = 0; j < 8; ++j) y[j] = merge_logit(c[j], u[j], s, inv_T);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) y[j] = __fmul_rn(c[j], inv_T);
  }
}

// Shared-memory layout (dynamic).  `work` is a 16 KB-or-larger region used as the histogram during
// selection and as id bitmap + per-word prefix during ordering; it also backs the generic fallback.
struct StreamSmem {
  uint64_t* full;        // [n_stages]
  uint64_t* empty;       // [n_stages]
  unsigned char* ring;   // [n_stages][2][kStageBytesPerArray]
  uint32_t* work;        // max(kHistBins, 2 * vwords) words
  Candidate* lists;      // [kLaneListCap][NT] interleaved per-thread lists
  Candidate* overflow;   // [kOverflowCap]
  int32_t* st_ids;       // [kStageKcapMax]
  float* st_vals;        // [kStageKcapMax]
  uint64_t* scan;        // group scratch
  int* ctl;              // control words
};
enum { kCtlOverflowCount = 0, kCtlAbort = 1, kCtlBin = 2, kCtlAbove = 3, kCtlBinCount = 4, kCtlThrId = 5,
       kCtlThrY = 6, kCtlPtok = 7, kCtlGather = 8, kCtlWords = 16 };

__host__ __device__ inline size_t stream_smem_bytes(int n_stages, int NT, int vwords) {
  size_t work_words = (size_t)(2 * vwords > kHistBins ? 2 * vwords : kHistBins);
  size_t b = 0;
  b += 2 * (size_t)n_stages * 8;
  b = (b + 127) & ~(size_t)127;
  b += (size_t)n_stages * 2 * kStageBytesPerArray;
  b += work_words * 4;
  b += (size_t)kLaneListCap * NT * sizeof(Candidate);
  b += (size_t)kOverflowCap * sizeof(Candidate);
  b += (size_t)kStageKcapMax * 8;
  b += (2 * 32 + 8) * 8;
  b += kCtlWords * 4;
  return b + 128;
}

template <int NT>
__device__ __forceinline__ StreamSmem carve_smem(unsigned char* base, int n_stages, int vwords) {
  StreamSmem s;
  uintptr_t p = (reinterpret_cast<uintptr_t>(base) + 127) & ~(uintptr_t)127;
  s.full = reinterpret_cast<uint64_t*>(p);
  s.empty = s.full + n_stages;
  p += 2 * (size_t)n_stages * 8;
  p = (p + 127) & ~(uintptr_t)127;
  s.ring = reinterpret_cast<unsigned char*>(p);
  p += (size_t)n_stages * 2 * kStageBytesPerArray;
  s.work = reinterpret_cast<uint32_t*>(p);
  p += (size_t)(2 * vwords > kHistBins ? 2 * vwords : kHistBins) * 4;
  s.lists = reinterpret_cast<Candidate*>(p);
  p += (size_t)kLaneListCap * NT * sizeof(Candidate);
  s.overflow = reinterpret_cast<Candidate*>(p);
  p += (size_t)kOverflowCap * sizeof(Candidate);
  s.st_ids = reinterpret_cast<int32_t*>(p);
  p += (size_t)kStageKcapMax * 4;
  s.st_vals = reinterpret_cast<float*>(p);
  p += (size_t)kStageKcapMax * 4;
  s.scan = reinterpret_cast<uint64_t*>(p);
  p += (2 * 32 + 8) * 8;
  s.ctl = reinterpret_cast<int*>(p);
  return s;
}

// Largest bin b with (number of entries in bins > b) < target <= (number in bins >= b); the count above
// it goes to ctl[kCtlAbove], the bin's own count to ctl[kCtlBinCount].  Writes bin -1 when the histogram
// holds fewer than `target` entries.  All NT threads call it; hist has kHistBins counters.
template <int NT, int BAR>
__device__ __forceinline__ void find_rank_bin(const uint32_t* hist, uint32_t target, int tid, uint64_t* scratch,
                                              int* ctl) {
  constexpr int PER = kHistBins / NT;
  static_assert(kHistBins % NT == 0, "bins must divide evenly");
  // thread t owns bins (from the top) kHistBins-1 - PER*t - j, j = 0..PER-1
  uint32_t c[PER], sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    c[j] = hist[kHistBins - 1 - PER * tid - j];
    sum += c[j];
  }
  if (tid == 0) ctl[kCtlBin] = -1;
  uint32_t total;
  uint32_t above = group_exclusive_scan<NT, BAR, uint32_t>(sum, tid, scratch, &total);
  if (above < target && target <= above + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (above < target && target <= above + c[j]) {
        ctl[kCtlBin] = kHistBins - 1 - PER * tid - j;
        ctl[kCtlAbove] = (int)above;
        ctl[kCtlBinCount] = (int)c[j];
      }
      above += c[j];
    }
  }
  group_sync<NT, BAR>();
}

// One warp's share of a staged tile set: append every element with y >= tau0 to the thread's list.
template <int DTYPE>
__device__ __forceinline__ void filter_tile(const unsigned char* ctile, const unsigned char* utile, bool has_u,
                                            int lane, float s, float inv_T, float tau0, int id_base,
                                            Candidate*& cursor, Candidate* limit, int list_stride,
                                            Candidate* overflow, int* ctl) {
  float y[8];
  tile_y8<DTYPE>(ctile, utile, has_u, lane, s, inv_T, y);
  if (cursor + 8 * list_stride <= limit) {
    // room for all eight: branch-free predicated appends
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (y[j] >= tau0) {
        *cursor = Candidate{y[j], id_base + tile_elem<DTYPE>(lane, j)};
        cursor += list_stride;
      }
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (y[j] >= tau0) {
        const Candidate cd{y[j], id_base + tile_elem<DTYPE>(lane, j)};
        if (cursor < limit) {
          *cursor = cd;
          cursor += list_stride;
        } else {
          const int o = atomicAdd(&ctl[kCtlOverflowCount], 1);
          if (o < kOverflowCap) overflow[o] = cd;
        }
      }
    }
  }
}

// Visit every candidate of the calling thread: its own list, then a strided share of the spill list.
template <int NT, typename F>
__device__ __forceinline__ void for_each_candidate(const StreamSmem& sm, int tid, int my_count, int n_over, F f) {
  for (int e = 0; e < my_count; ++e) f(sm.lists[e * NT + tid]);
  for (int o = tid; o < n_over; o += NT) f(sm.overflow[o]);
}

template <int DTYPE, int NCW>
__global__ void __launch_bounds__(NCW * 32 + 32, 1) rows_stream_kernel(const RowArgs a, const StreamCfg cfg) {
  constexpr int NT = NCW * 32;
  constexpr int BAR = 1;
  using TR = StreamTraits<DTYPE>;
  constexpr int TPS = TR::kTilesPerStage;
  extern __shared__ unsigned char smem_raw[];
  StreamSmem sm = carve_smem<NT>(smem_raw, cfg.n_stages, cfg.vwords);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int NS = cfg.n_stages;
  const bool has_u = a.uncond != nullptr;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], NCW);
    }
    sm.ctl[kCtlAbort] = 0;
    fence_barrier_init();
  }
  __syncthreads();

  const RowSchedule sched(a.V, cfg.sample_stride, TPS);
  const int rows = a.B * a.W;

  if (warp == NCW) {
    // =============================== producer warp ===============================
    uint32_t it = 0;  // stages issued so far by this CTA
    bool ok = true;
    for (int row = blockIdx.x; row < rows && ok; row += gridDim.x) {
      const int b = row / a.W, i = row - b * a.W;
      const int L = a.win_len ? min(max(a.win_len[b], 0), a.W) : a.W;
      if (i >= L) continue;
      const int64_t off = (int64_t)b * a.stride_b + (int64_t)i * a.stride_w;
      const unsigned char* gc = static_cast<const unsigned char*>(a.cond) + off * TR::kElemBytes;
      const unsigned char* gu = has_u ? static_cast<const unsigned char*>(a.uncond) + off * TR::kElemBytes : nullptr;
      for (int s = 0; s < sched.stages; ++s, ++it) {
        const int slot = it % NS;
        const uint32_t use = it / NS;
        if (use > 0) ok = mbar_wait(&sm.empty[slot], (use - 1) & 1u);
        ok = __all_sync(0xffffffffu, ok) && (*reinterpret_cast<volatile int*>(&sm.ctl[kCtlAbort]) == 0);
        if (!ok) break;
        const int nt = sched.stage_tiles(s, TPS);
        unsigned char* dst_c = sm.ring + (size_t)slot * TR::kStageBytes;
        unsigned char* dst_u = dst_c + kStageBytesPerArray;
        if (lane == 0) mbar_arrive_expect_tx(&sm.full[slot], (uint32_t)nt * TR::kTileBytes * (has_u ? 2u : 1u));
        __syncwarp();
        if (s == 0) {
          // sample tiles are isolated: one copy per tile, spread over the lanes
          for (int j = lane; j < nt; j += 32) {
            const size_t goff = (size_t)j * sched.ss * TR::kTileBytes;
            bulk_g2s(dst_c + (size_t)j * TR::kTileBytes, gc + goff, TR::kTileBytes, &sm.full[slot]);
            if (has_u) bulk_g2s(dst_u + (size_t)j * TR::kTileBytes, gu + goff, TR::kTileBytes, &sm.full[slot]);
          }
        } else {
          // tail tiles come in runs of SS-1 contiguous tiles: lane r copies the r-th run of the stage
          const int t0 = TPS * (s - 1), t1 = t0 + nt, rl = sched.ss - 1;
          const int first_run = t0 / rl;
          const int run = first_run + lane;
          const int ta = max(run * rl, t0), tb = min((run + 1) * rl, t1);
          if (ta < tb) {
            const int g = run * sched.ss + 1 + (ta - run * rl);
            const uint32_t bytes = (uint32_t)(tb - ta) * TR::kTileBytes;
            const size_t goff = (size_t)g * TR::kTileBytes, soff = (size_t)(ta - t0) * TR::kTileBytes;
            bulk_g2s(dst_c + soff, gc + goff, bytes, &sm.full[slot]);
            if (has_u) bulk_g2s(dst_u + soff, gu + goff, bytes, &sm.full[slot]);
          }
        }
      }
    }
    // drain: every stage this warp armed must have landed before the CTA may exit
    {
      const uint32_t first = it > (uint32_t)NS ? it - NS : 0;
      for (uint32_t k = first; k < it; ++k) mbar_wait(&sm.full[k % NS], (k / NS) & 1u);
      if (!ok && lane == 0) sm.ctl[kCtlAbort] = 1;
    }
    return;
  }

  // ================================= consumer warps =================================
  const int tid = threadIdx.x;  // 0 .. NT-1
  Candidate* const list_begin = sm.lists + tid;
  Candidate* const list_limit = sm.lists + (size_t)kLaneListCap * NT;
  uint32_t it = 0;
  bool aborted = false;
  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
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
    if (aborted) {
      if (tid == 0) {
        a.out_cnt[row] = 0;
        *rs = RowScratch{0.0f, -1, 0.0f, kRowStatusTimeout};
      }
      continue;
    }
    const int kcap = a.kcap;
    Candidate* cursor = list_begin;
    if (tid == 0) {
      sm.ctl[kCtlOverflowCount] = 0;
      sm.ctl[kCtlGather] = 0;
    }

    // ---------------- stage 0: the sample fixes tau0, then is filtered like any other stage ----------------
    for (int j = tid; j < kHistBins; j += NT) sm.work[j] = 0;
    group_sync<NT, BAR>();
    const int slot0 = it % NS;
    if (!mbar_wait(&sm.full[slot0], (it / NS) & 1u)) aborted = true;
    aborted = group_any<NT, BAR>(aborted);
    if (aborted) {
      if (tid == 0) {
        sm.ctl[kCtlAbort] = 1;
        a.out_cnt[row] = 0;
        *rs = RowScratch{0.0f, -1, 0.0f, kRowStatusTimeout};
      }
      continue;
    }
    const unsigned char* st_c = sm.ring + (size_t)slot0 * TR::kStageBytes;
    const unsigned char* st_u = st_c + kStageBytesPerArray;
    const int nt0 = sched.sample_tiles;
    for (int j = warp; j < nt0; j += NCW) {
      float y[8];
      tile_y8<DTYPE>(st_c + (size_t)j * TR::kTileBytes, st_u + (size_t)j * TR::kTileBytes, has_u, lane, a.s, a.inv_T, y);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float yc = canonical(y[e]);
        atomicAdd(&sm.work[float_key(yc) >> 20], 1u);
      }
    }
    group_sync<NT, BAR>();
    find_rank_bin<NT, BAR>(sm.work, (uint32_t)cfg.sample_rank, tid, sm.scan, sm.ctl);
    float tau0;
    {
      const int bin = sm.ctl[kCtlBin];
      // lower edge of the bin as a float; bin <= 0x7ff covers keys of negative floats
      const float lowest = -3.402823466e38f;  // every finite value is a candidate
      if (bin < 0) tau0 = lowest;
      else {
        const uint32_t key = (uint32_t)bin << 20;
        const uint32_t bits = (key & 0x80000000u) ? (key & 0x7fffffffu) : ~key;
        tau0 = __uint_as_float(bits);
        if (!(tau0 >= lowest)) tau0 = lowest;  // edge fell on -inf or into the NaN patterns
      }
    }
    for (int j = warp; j < nt0; j += NCW)
      filter_tile<DTYPE>(st_c + (size_t)j * TR::kTileBytes, st_u + (size_t)j * TR::kTileBytes, has_u, lane, a.s, a.inv_T,
                         tau0, sched.global_tile(0, j, TPS) * kTileElems, cursor, list_limit, NT, sm.overflow, sm.ctl);
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[slot0]);
    ++it;

    // ---------------- remaining stages ----------------
    for (int s = 1; s < sched.stages; ++s, ++it) {
      const int slot = it % NS;
      if (!mbar_wait(&sm.full[slot], (it / NS) & 1u)) {
        aborted = true;
        sm.ctl[kCtlAbort] = 1;
      }
      const unsigned char* sc = sm.ring + (size_t)slot * TR::kStageBytes;
      const unsigned char* su = sc + kStageBytesPerArray;
      const int nt = sched.stage_tiles(s, TPS);
      if (!aborted)
        for (int j = warp; j < nt; j += NCW)
          filter_tile<DTYPE>(sc + (size_t)j * TR::kTileBytes, su + (size_t)j * TR::kTileBytes, has_u, lane, a.s, a.inv_T,
                             tau0, sched.global_tile(s, j, TPS) * kTileElems, cursor, list_limit, NT, sm.overflow,
                             sm.ctl);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[slot]);
    }
    aborted = group_any<NT, BAR>(aborted);
    if (aborted) {
      if (tid == 0) {
        a.out_cnt[row] = 0;
        *rs = RowScratch{0.0f, -1, 0.0f, kRowStatusTimeout};
      }
      continue;
    }

    // ---------------- exact top-K among the candidates ----------------
    const int my_count = (int)((cursor - list_begin) / NT);
    const int n_over_raw = sm.ctl[kCtlOverflowCount];
    const int n_over = min(n_over_raw, kOverflowCap);
    uint32_t n_total;
    group_exclusive_scan<NT, BAR, uint32_t>((uint32_t)my_count, tid, sm.scan, &n_total);
    n_total += (uint32_t)n_over;
    bool fallback = (n_over_raw > kOverflowCap) || (n_total < (uint32_t)kcap) || (kcap > kStageKcapMax);

    float vmax = __int_as_float(0xff800000);
    if (!fallback) {
      for_each_candidate<NT>(sm, tid, my_count, n_over, [&](const Candidate& c) { vmax = fmaxf(vmax, c.y); });
      vmax = group_max_f32<NT, BAR>(vmax, tid, sm.scan);
    }
    float thr_y = 0.0f;
    int thr_id = 0;
    if (!fallback) {
      // linear bins over [tau0, vmax]; monotone in y, so higher bins hold strictly larger values
      const float range = __fsub_rn(vmax, tau0);
      const float scale = range > 0.0f ? __fdiv_rn((float)kHistBins * 0.999f, range) : 0.0f;
      auto bin_of = [&](float y) {
        const int q = __float2int_rd(__fmul_rn(__fsub_rn(canonical(y), tau0), scale));
        return min(max(q, 0), kHistBins - 1);
      };
      for (int j = tid; j < kHistBins; j += NT) sm.work[j] = 0;
      group_sync<NT, BAR>();
      for_each_candidate<NT>(sm, tid, my_count, n_over, [&](const Candidate& c) { atomicAdd(&sm.work[bin_of(c.y)], 1u); });
      group_sync<NT, BAR>();
      find_rank_bin<NT, BAR>(sm.work, (uint32_t)kcap, tid, sm.scan, sm.ctl);
      const int tbin = sm.ctl[kCtlBin];
      const int need = kcap - sm.ctl[kCtlAbove];  // members of the threshold bin that survive
      const int nbin = sm.ctl[kCtlBinCount];
      if (tbin < 0 || nbin > kBinListCap) fallback = true;
      if (!fallback) {
        // gather the threshold bin and rank its members by (y descending, id ascending)
        Candidate* binlist = reinterpret_cast<Candidate*>(sm.st_ids);  // staging is free until ordering
        static_assert(kBinListCap * sizeof(Candidate) <= kStageKcapMax * 8, "bin list must fit the staging area");
        for_each_candidate<NT>(sm, tid, my_count, n_over, [&](const Candidate& c) {
          if (bin_of(c.y) == tbin) binlist[atomicAdd(&sm.ctl[kCtlGather], 1)] = Candidate{canonical(c.y), c.id};
        });
        group_sync<NT, BAR>();
        for (int x = tid; x < nbin; x += NT) {
          const Candidate me = binlist[x];
          int rank = 0;
          for (int z = 0; z < nbin; ++z) {
            const Candidate o = binlist[z];
            rank += (o.y > me.y || (o.y == me.y && o.id < me.id)) ? 1 : 0;
          }
          if (rank == need - 1) {
            sm.ctl[kCtlThrY] = __float_as_int(me.y);
            sm.ctl[kCtlThrId] = me.id;
          }
        }
        group_sync<NT, BAR>();
        thr_y = __int_as_float(sm.ctl[kCtlThrY]);
        thr_id = sm.ctl[kCtlThrId];
      }
    }
    if (fallback) {
      // exact any-shape path from global memory (the row is still in L2)
      row_generic<DTYPE, NT, BAR>(a, row, tid, *reinterpret_cast<GenericSmem*>(sm.work));
      continue;
    }
    auto survives = [&](const Candidate& c) {
      const float y = canonical(c.y);
      return y > thr_y || (y == thr_y && c.id <= thr_id);
    };

    // ---------------- ascending-id order through a bitmap over token ids ----------------
    uint32_t* bitmap = sm.work;
    uint32_t* wprefix = sm.work + cfg.vwords;
    for (int j = tid; j < cfg.vwords; j += NT) bitmap[j] = 0;
    group_sync<NT, BAR>();
    for_each_candidate<NT>(sm, tid, my_count, n_over, [&](const Candidate& c) {
      if (survives(c)) atomicOr(&bitmap[c.id >> 5], 1u << (c.id & 31));
    });
    group_sync<NT, BAR>();
    {
      // exclusive prefix of the per-word popcounts; each thread owns a contiguous run of words
      const int per = (cfg.vwords + NT - 1) / NT;
      const int w0 = tid * per, w1 = min(w0 + per, cfg.vwords);
      uint32_t sum = 0;
      for (int w = w0; w < w1; ++w) sum += __popc(bitmap[w]);
      uint32_t total;
      uint32_t run = group_exclusive_scan<NT, BAR, uint32_t>(sum, tid, sm.scan, &total);
      for (int w = w0; w < w1; ++w) {
        wprefix[w] = run;
        run += __popc(bitmap[w]);
      }
      if (tid == 0) sm.ctl[kCtlPtok] = 0;
      group_sync<NT, BAR>();
      if (total != (uint32_t)kcap) {  // cannot happen; keep the result exact anyway
        row_generic<DTYPE, NT, BAR>(a, row, tid, *reinterpret_cast<GenericSmem*>(sm.work));
        continue;
      }
    }
    // ---------------- softmax numerators into id order ----------------
    float zpart = 0.0f;
    for_each_candidate<NT>(sm, tid, my_count, n_over, [&](const Candidate& c) {
      if (survives(c)) {
        const int pos = (int)(wprefix[c.id >> 5] + __popc(bitmap[c.id >> 5] & ((1u << (c.id & 31)) - 1u)));
        const float e = exp_diff(canonical(c.y), vmax);
        sm.st_ids[pos] = c.id;
        sm.st_vals[pos] = e;
        zpart += e;
      }
    });
    const float Z = group_sum_f32<NT, BAR>(zpart, tid, sm.scan);
    const int draft = a.drafts ? a.drafts[row] : -1;
    int32_t* out_ids = a.out_ids + (size_t)row * kcap;
    float* out_vals = a.out_vals + (size_t)row * kcap;
    for (int k = tid; k < kcap; k += NT) {
      const float p = __fdiv_rn(sm.st_vals[k], Z);
      const int id = sm.st_ids[k];
      sm.st_vals[k] = p;
      out_ids[k] = id;
      out_vals[k] = p;
      if (id == draft) sm.ctl[kCtlPtok] = __float_as_int(p);
    }
    group_sync<NT, BAR>();
    // ---------------- the row's own draw from p_i ----------------
    const int pos = (a.pos_base ? a.pos_base[b] : 0) + i;
    const int iter = a.iteration ? a.iteration[b] : a.iteration0;
    const Philox4 rnd =
        philox4x32_10((uint32_t)pos, (uint32_t)(a.seq_base + b), (uint32_t)iter, (uint32_t)a.purpose, a.seed_lo, a.seed_hi);
    int k = group_icdf<NT, BAR>([&](int kk) { return fixed_weight(sm.st_vals[kk]); }, kcap, random64(rnd), tid, sm.scan);
    if (k < 0) k = 0;
    if (tid == 0) {
      a.out_cnt[row] = kcap;
      *rs = RowScratch{__int_as_float(sm.ctl[kCtlPtok]), sm.st_ids[k], sm.st_vals[k], 0};
    }
    group_sync<NT, BAR>();
  }
}

}  // namespace sjd

// Host side of the C ABI declared in include/sjd.h: argument checks and kernel launches.
// Nothing here allocates, frees or synchronises.
#include "../../include/sjd.h"

#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "device_once.h"
#include "device_utils.cuh"
#include "row_kernels.cuh"
#include "rows_pipeline.cuh"
#include "rows_ranges.cuh"
#include "verify_kernel.cuh"
#include "advance_kernel.cuh"

#include <cmath>

namespace {

thread_local char g_cuda_error[256] = "";
std::atomic<uint64_t> g_launches{0};

int cuda_fail(cudaError_t e, const char* what) {
  std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(e));
  return SJD_ERR_CUDA;
}

constexpr int kGenericThreads = 512;
constexpr int kVerifyThreads = 512;

int current_device() {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

// SM count of the current device (cached per device ordinal).
int sm_count() {
  static sjd::DeviceValue cache;
  const int dev = current_device();
  const int n = cache.get(dev, [dev] {
    int v = 0;
    return (dev >= 0 && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) ? v : 0;
  });
  return n > 0 ? n : 148;
}

// The opt-in to more than 48 KB of dynamic shared memory belongs to the (device, kernel) pair: it is set
// once per device for each kernel instantiation (`once` is that instantiation's record).
template <typename Kern>
cudaError_t allow_large_smem(Kern kern, sjd::DeviceOnce& once, int bytes) {
  cudaError_t err = cudaSuccess;
  once.run_once(current_device(), [&] {
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return err == cudaSuccess ? 0 : 1;
  });
  return err;
}

constexpr int kFilterWarps = 8;
constexpr int kFinisherWarps = 8;
constexpr int kMaxStages = 12;
constexpr size_t kSmemLimit = 227u * 1024u;

// Decide whether the single-pass pipelined kernel can take this shape, and with which sampling
// parameters.  The sample is every SS-th 256-element tile of a row; its rank-m value (from the top)
// becomes the candidate threshold.  m is chosen 4.5 standard deviations above K/SS (sample_rank), so that
// a row with exchangeable entries almost never fails to deliver K candidates (such a row is redone by the
// any-shape path, never answered wrongly).  The on-chip lists must hold the expected number of
// candidates with a margin: four standard deviations for the row's total, and for the share of one
// filter thread (a Poisson count) a tail below 1e-6.
// Rank m of the sample element that serves as the first threshold, for an expected a = kcap / S of the row's
// kcap largest inside a sample of one S-th of the row.  The number of those that really fall in the sample
// is at most Poisson(a)-distributed (drawing without replacement only narrows it), so m = a + z sqrt(m),
// i.e. sqrt(m) = z/2 + sqrt(z^2/4 + a), leaves the threshold above the true one (too few candidates, the
// row redone by the any-shape path at many times the cost) with a probability below 4e-6 per row at z = 4.5.
int sample_rank(double a, double z = 4.5) {
  const double root = z / 2 + std::sqrt(z * z / 4 + a);
  return (int)std::ceil(root * root);
}

bool plan_pipeline(const sjd_params* P, int kcap, sjd::PipeCfg* cfg, size_t* smem) {
  const int V = P->V;
  if (kcap > sjd::kKcapMax || V % sjd::kTileElems != 0) return false;
  const int tile_bytes = sjd::kTileElems * (P->logits_dtype == SJD_F32 ? 4 : 2);
  const int tps = sjd::kStageArrayBytes / tile_bytes;
  const int tiles = V / sjd::kTileElems;
  const int vwords = V / 32;
  if (tiles > sjd::kItersMax * kFilterWarps) return false;
  for (int ss : {8, 16, 32}) {
    if (tiles % ss != 0) continue;
    const int sample_tiles = tiles / ss, tail_tiles = tiles - sample_tiles;
    const int sample_stages = (sample_tiles + tps - 1) / tps;
    // tiles of filter warp 0 per row (the most any warp gets), four hit bits each
    int iters0 = 0;
    for (int left = sample_tiles; left > 0; left -= tps) iters0 += ((left < tps ? left : tps) + kFilterWarps - 1) / kFilterWarps;
    for (int left = tail_tiles; left > 0; left -= tps) iters0 += ((left < tps ? left : tps) + kFilterWarps - 1) / kFilterWarps;
    const int mask_words = (4 * iters0 + 31) / 32;
    if (iters0 > sjd::kItersMax || mask_words > sjd::kMaskWordsMax) continue;
    const size_t fixed = sjd::pipe_smem_fixed_bytes(kFilterWarps, vwords, mask_words);
    if (fixed + (size_t)(sample_stages + 3) * 2 * sjd::kStageArrayBytes > kSmemLimit) continue;
    int ns = (int)((kSmemLimit - fixed) / (2 * (size_t)sjd::kStageArrayBytes));
    if (ns > kMaxStages) ns = kMaxStages;
    const int n_sample = V / ss;
    const double a = (double)kcap / ss;
    const int m = sample_rank(a);
    if (m > n_sample / 2 || m > 32 * sample_tiles) continue;  // the rank must exist among the group maxima too
    const double mean = (double)m * ss, sd = (double)ss * std::sqrt((double)m);
    if (mean + 4.0 * sd > (double)sjd::kDenseCap) continue;
    // sample pairs are kept against a floor somewhat below the threshold: about 2m more entries
    const double per_thread = (mean + 2.0 * m) / (32.0 * kFilterWarps);
    if (per_thread + 5.0 * std::sqrt(per_thread) + 1.0 > (double)(sjd::kListCap - 4)) continue;
    cfg->sample_stride = ss;
    cfg->sample_rank = m;
    cfg->n_stages = ns;
    cfg->vwords = vwords;
    cfg->mask_words = mask_words;
    *smem = sjd::pipe_smem_bytes(ns, kFilterWarps, vwords, mask_words);
    return true;
  }
  return false;
}

// ---- the kernel with one id range per filter thread (rows_ranges.cuh) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime (no link against the driver library); nullptr when unavailable.
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess ||
        qr != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Same sampling rule as plan_pipeline; the sample is stage 0, i.e. 1/S of the row.
bool plan_ranges(const sjd_params* P, int kcap, sjd::RangeCfg* cfg, size_t* smem, bool need_encoder = true) {
  const int V = P->V;
  const int es = P->logits_dtype == SJD_F32 ? 4 : 2;
  const int bw = 64 / es;  // elements per stage and range
  if (kcap > sjd::kKcapMax || V % sjd::kRangeThreads != 0) return false;
  const int R = V / sjd::kRangeThreads;
  if (R % bw != 0) return false;
  const int S = R / bw;
  if (S < 2 || S > 16) return false;
  // all rows must lie at one pitch: row r = b W + i starts at r * stride_w
  if (P->B > 1 && P->stride_b != (int64_t)P->W * P->stride_w) return false;
  if ((int64_t)P->B * P->W >= (1ll << 31)) return false;
  const int mask_words = (R / 2 + 31) / 32;
  if (mask_words > sjd::kMaskWordsMax) return false;
  const int n_sample = sjd::kRangeThreads * bw;
  const double a = (double)kcap / S;
  int m = sample_rank(a);
  if (m > n_sample / 2) return false;
  // The element rank m can be taken as a rank among the maxima of the sample's groups of eight (see the
  // sampler): directly while at most a tenth of the sample lies above the threshold.  Up to a fifth the group
  // maxima still resolve the rank, but up to 1.6 times less sharply than the elements would: a margin of 6.5
  // instead of 4.5 standard deviations keeps the row at least as safe.  Beyond that every element is binned.
  bool by_groups = m <= n_sample / 8 && (double)m / n_sample <= 0.10;
  if (!by_groups) {
    const int m_wide = sample_rank(a, 6.5);
    if ((double)m_wide / n_sample <= 0.20) {
      m = m_wide;
      by_groups = true;
    }
  }
  const int sample_all = m > n_sample / 8 ? 1 : 0;  // the rank must exist among what an element-wise first pass bins
  // candidates of a row: m S on average; pairs of neighbours with at least one candidate: a little fewer
  const double cand = (double)m * S, cand_sd = (double)S * std::sqrt((double)m);
  const double thin = 1.0 - 0.5 * cand / V;
  if ((cand + 5.0 * cand_sd) * thin > (double)sjd::kRangePairCap) return false;
  // pair entries per filter thread: a Poisson count; its list must hold it with a tail below 1e-6
  const double per_thread = cand * thin / sjd::kRangeThreads;
  if (per_thread + 5.0 * std::sqrt(per_thread) + 1.0 > (double)(sjd::kRangeListCap - 4)) return false;
  if (need_encoder && encode_tiled_fn() == nullptr) return false;
  cfg->sample_rank = m;
  cfg->sample_all = sample_all;
  {
    const double p = (double)m / n_sample, groups = n_sample / 8.0;
    cfg->group_rank = by_groups ? (int)std::ceil(groups * (1.0 - std::pow(1.0 - p, 8.0))) : 0;
  }
  cfg->stages = S;
  cfg->range_len = R;
  cfg->mask_words = mask_words;
  cfg->row_begin = 0;
  cfg->row_end = P->B * P->W;
  *smem = sjd::range_smem_bytes(mask_words);
  return *smem <= kSmemLimit;
}

// Tensor map over one logits array: dims {R ids, 256 ranges, rows}, box {64 bytes, 256, 1}, 64-byte swizzle.
// L2 promotion stays at the box's own 64 bytes per range: wider promotion fetches the neighbouring stages
// early, and measured slower (128 bytes: +1.6 us, 256 bytes: +5 us on the headline workload) than the kernel's
// own prefetch one ring depth ahead.
bool make_range_map(CUtensorMap* map, const void* base, const sjd_params* P, const sjd::RangeCfg& cfg) {
  const int es = P->logits_dtype == SJD_F32 ? 4 : 2;
  const cuuint64_t dims[3] = {(cuuint64_t)cfg.range_len, (cuuint64_t)sjd::kRangeThreads, (cuuint64_t)P->B * (cuuint64_t)P->W};
  const cuuint64_t strides[2] = {(cuuint64_t)cfg.range_len * es, (cuuint64_t)P->stride_w * es};
  const cuuint32_t box[3] = {(cuuint32_t)(64 / es), (cuuint32_t)sjd::kRangeThreads, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = encode_tiled_fn()(map, P->logits_dtype == SJD_BF16  ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                       : P->logits_dtype == SJD_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                                    : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                       3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                       CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_64B,
                                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Launch as a programmatic dependent of the stream's previous kernel: when that kernel allows it (ours do
// near their end), this grid's blocks are placed and set up early and wait inside the kernel
// (grid_dependency_wait) until the previous kernel has completed.  After a kernel that does not take part,
// an event or a copy this is an ordinary launch.
template <typename... KArgs, typename... Args>
cudaError_t launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool dependent,
                         Args&&... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = dependent ? 1 : 0;
  return cudaLaunchKernelEx(&lc, kern, std::forward<Args>(args)...);
}

constexpr int kSamplerWarps = 3;
constexpr int kRangeFinisherWarps = 16;

// One kernel per logits type and per combination of (guidance given, temperature applied, thresholds by
// group maxima): each holds only the code its launch runs, which matters because the roles' code does not fit
// the instruction caches comfortably.
template <int DTYPE, bool HAS_U, bool HAS_T, bool BY_GROUPS>
cudaError_t launch_ranges_as(const sjd::RowArgs& ra, const sjd::RangeCfg& cfg, const CUtensorMap& mc, const CUtensorMap& mu,
                             size_t smem, int grid, cudaStream_t st) {
  auto kern = sjd::rows_ranges_kernel<DTYPE, kRangeFinisherWarps, kSamplerWarps, HAS_U, HAS_T, BY_GROUPS>;
  static sjd::DeviceOnce configured;  // per instantiation
  const cudaError_t e = allow_large_smem(kern, configured, (int)kSmemLimit);
  if (e != cudaSuccess) return e;
  return launch_after(kern, dim3((unsigned)grid), dim3((8 + kRangeFinisherWarps + kSamplerWarps + 1) * 32), smem, st, true, ra,
                      cfg, mc, mu);
}

template <int DTYPE>
cudaError_t launch_ranges(const sjd::RowArgs& ra, const sjd::RangeCfg& cfg, const CUtensorMap& mc, const CUtensorMap& mu,
                          size_t smem, int grid, cudaStream_t st) {
  const int which = (ra.uncond != nullptr ? 4 : 0) | (ra.inv_T != 1.0f ? 2 : 0) | (cfg.group_rank > 0 ? 1 : 0);
  switch (which) {
    case 0: return launch_ranges_as<DTYPE, false, false, false>(ra, cfg, mc, mu, smem, grid, st);
    case 1: return launch_ranges_as<DTYPE, false, false, true>(ra, cfg, mc, mu, smem, grid, st);
    case 2: return launch_ranges_as<DTYPE, false, true, false>(ra, cfg, mc, mu, smem, grid, st);
    case 3: return launch_ranges_as<DTYPE, false, true, true>(ra, cfg, mc, mu, smem, grid, st);
    case 4: return launch_ranges_as<DTYPE, true, false, false>(ra, cfg, mc, mu, smem, grid, st);
    case 5: return launch_ranges_as<DTYPE, true, false, true>(ra, cfg, mc, mu, smem, grid, st);
    case 6: return launch_ranges_as<DTYPE, true, true, false>(ra, cfg, mc, mu, smem, grid, st);
    default: return launch_ranges_as<DTYPE, true, true, true>(ra, cfg, mc, mu, smem, grid, st);
  }
}

template <int DTYPE>
cudaError_t launch_pipeline(const sjd::RowArgs& ra, const sjd::PipeCfg& cfg, size_t smem, int grid, cudaStream_t st) {
  auto kern = sjd::rows_pipeline_kernel<DTYPE, kFilterWarps, kFinisherWarps>;
  static sjd::DeviceOnce configured;  // per instantiation
  const cudaError_t e = allow_large_smem(kern, configured, (int)kSmemLimit);
  if (e != cudaSuccess) return e;
  return launch_after(kern, dim3((unsigned)grid), dim3((kFilterWarps + kFinisherWarps + 1) * 32), smem, st, true, ra, cfg);
}

// Scratch of sjd_step_static(): lives in the library's device image, so every GPU that loads the library
// holds these bytes until the process exits.  Sized for SJD_STATIC_MAX_ROWS rows of RowScratch.
constexpr size_t kStaticScratchBytes = (((size_t)SJD_STATIC_MAX_ROWS * sizeof(sjd::RowScratch) + 256) + 255) & ~(size_t)255;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

using sjd::kMaxDevices;
std::mutex g_static_mutex;
void* g_static_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

// Device address of the static scratch on the CURRENT device.  In host code the symbol's name is only a
// handle; the address a kernel can use comes from cudaGetSymbolAddress(), asked once per device.
int static_scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  if (dev < 0 || dev >= kMaxDevices) return SJD_ERR_CAPACITY;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
    if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 255u) != 0) return SJD_ERR_WORKSPACE;
    g_static_scratch_addr[dev] = p;
  }
  *out = g_static_scratch_addr[dev];
  return SJD_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_probs(const sjd_probs* p) {
  if (!p || !p->tok_prob || !p->ids || !p->vals || !p->cnt) return SJD_ERR_NULL;
  return SJD_OK;
}

}  // namespace

extern "C" {

int sjd_version(void) { return SJD_VERSION; }

const char* sjd_status_string(int code) {
  switch (code) {
    case SJD_OK: return "ok";
    case SJD_ERR_NULL: return "a required pointer is NULL";
    case SJD_ERR_SHAPE: return "bad shape: need B >= 0, 1 <= W <= SJD_W_MAX, V >= 8 and V % 8 == 0, top_k >= 1";
    case SJD_ERR_ALIGN: return "logits base address or strides are not 16-byte aligned";
    case SJD_ERR_DTYPE: return "unknown logits dtype";
    case SJD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SJD_ERR_STRUCT: return "struct_size does not match this library";
    case SJD_ERR_CUDA: return "CUDA runtime error";
    case SJD_ERR_CAPACITY: return "problem exceeds the fixed capacity of this entry point";
    default: return "unknown status";
  }
}

const char* sjd_last_cuda_error(void) { return g_cuda_error; }

uint64_t sjd_launch_count(void) { return g_launches.load(); }

#ifdef SJD_PHASE_TIMERS
// Diagnostic builds only: copies the 48 phase counters to `out` (host) after a device synchronisation and
// optionally clears them.
int sjd_phase_cycles_read(unsigned long long* out, int reset) {
  if (cudaDeviceSynchronize() != cudaSuccess) return SJD_ERR_CUDA;
  if (cudaMemcpyFromSymbol(out, sjd::g_phase_cycles, sizeof(unsigned long long) * 48) != cudaSuccess) return SJD_ERR_CUDA;
  if (reset) {
    unsigned long long z[48] = {0};
    if (cudaMemcpyToSymbol(sjd::g_phase_cycles, z, sizeof(z)) != cudaSuccess) return SJD_ERR_CUDA;
  }
  return SJD_OK;
}
#endif

size_t sjd_workspace_bytes(const sjd_params* p) {
  if (!p || p->B < 0 || p->W < 1) return 0;
  const size_t rows = (size_t)p->B * (size_t)p->W;
  const size_t bytes = rows * sizeof(sjd::RowScratch) + 256;
  return (bytes + 255) & ~(size_t)255;
}

int sjd_step(const void* logits_cond, const void* logits_uncond, const int32_t* drafts, const sjd_probs* draft_probs,
             const sjd_params* P, uint64_t philox_seed, int32_t* out_accept_len, int32_t* out_tokens,
             sjd_probs* out_probs) {
  if (!P) return SJD_ERR_NULL;
  if (P->struct_size != (int32_t)sizeof(sjd_params)) return SJD_ERR_STRUCT;
  if (!logits_cond || !out_accept_len || !out_tokens) return SJD_ERR_NULL;
  if (check_probs(out_probs) != SJD_OK) return SJD_ERR_NULL;
  const bool draft_all = (P->flags & SJD_FLAG_DRAFT_ALL) != 0;
  if (!draft_all && (!drafts || check_probs(draft_probs) != SJD_OK)) return SJD_ERR_NULL;
  if (P->B < 0 || P->W < 1 || P->W > SJD_W_MAX || P->V < 8 || (P->V % 8) != 0 || P->top_k < 1) return SJD_ERR_SHAPE;
  if (P->logits_dtype != SJD_F32 && P->logits_dtype != SJD_BF16 && P->logits_dtype != SJD_F16) return SJD_ERR_DTYPE;
  const int64_t esize = P->logits_dtype == SJD_F32 ? 4 : 2;
  if (!aligned16(logits_cond) || (logits_uncond && !aligned16(logits_uncond)) || (P->stride_b * esize) % 16 != 0 ||
      (P->stride_w * esize) % 16 != 0 || P->stride_w < P->V || P->stride_b < 0)
    return SJD_ERR_ALIGN;
  if (!P->workspace || (reinterpret_cast<uintptr_t>(P->workspace) & 255u) != 0 ||
      P->workspace_bytes < sjd_workspace_bytes(P))
    return SJD_ERR_WORKSPACE;
  if (P->B == 0) return SJD_OK;

  cudaStream_t stream = static_cast<cudaStream_t>(P->stream);
  const int kcap = P->top_k < P->V ? P->top_k : P->V;
  const int rows = P->B * P->W;

  sjd::RowArgs ra;
  ra.cond = logits_cond;
  ra.uncond = logits_uncond;
  ra.stride_b = P->stride_b;
  ra.stride_w = P->stride_w;
  ra.B = P->B; ra.W = P->W; ra.V = P->V; ra.kcap = kcap;
  ra.s = P->cfg_scale;
  ra.inv_T = P->inv_temperature;
  ra.win_len = P->win_len;
  ra.pos_base = P->pos_base;
  ra.iteration = P->iteration;
  ra.iteration0 = P->iteration0;
  ra.seq_base = P->seq_base;
  ra.drafts = draft_all ? nullptr : drafts;
  ra.seed_lo = (uint32_t)(philox_seed & 0xffffffffu);
  ra.seed_hi = (uint32_t)(philox_seed >> 32);
  ra.purpose = draft_all ? sjd::kPurposeInit : sjd::kPurposeRedraft;
  ra.out_ids = out_probs->ids;
  ra.out_vals = out_probs->vals;
  ra.out_cnt = out_probs->cnt;
  ra.scratch = static_cast<sjd::RowScratch*>(P->workspace);

  if (P->ev_rows_begin) {
    const cudaError_t e = cudaEventRecord(static_cast<cudaEvent_t>(P->ev_rows_begin), stream);
    if (e != cudaSuccess) return cuda_fail(e, "event record");
  }
  {
    sjd::PipeCfg cfg;
    sjd::RangeCfg rcfg;
    size_t smem = 0;
    cudaError_t e;
    CUtensorMap map_c, map_u;
    const bool fast = !(P->flags & (SJD_FLAG_FORCE_GENERIC | SJD_FLAG_FORCE_TILES));
    if (fast && plan_ranges(P, kcap, &rcfg, &smem) && make_range_map(&map_c, logits_cond, P, rcfg) &&
        make_range_map(&map_u, logits_uncond ? logits_uncond : logits_cond, P, rcfg)) {
      // a CTA takes at most kRowsPerCta rows per launch: larger problems go in several launches
      const int per_launch = sjd::kRowsPerCta * sm_count();
      e = cudaSuccess;
      for (int r0 = 0; r0 < rows && e == cudaSuccess; r0 += per_launch) {
        rcfg.row_begin = r0;
        rcfg.row_end = r0 + per_launch < rows ? r0 + per_launch : rows;
        const int n = rcfg.row_end - r0;
        const int grid = n < sm_count() ? n : sm_count();
        e = P->logits_dtype == SJD_BF16  ? launch_ranges<1>(ra, rcfg, map_c, map_u, smem, grid, stream)
            : P->logits_dtype == SJD_F16 ? launch_ranges<2>(ra, rcfg, map_c, map_u, smem, grid, stream)
                                         : launch_ranges<0>(ra, rcfg, map_c, map_u, smem, grid, stream);
        if (e == cudaSuccess && r0 > 0) ++g_launches;
      }
    } else if (!(P->flags & SJD_FLAG_FORCE_GENERIC) && plan_pipeline(P, kcap, &cfg, &smem)) {
      const int grid = rows < sm_count() ? rows : sm_count();
      e = P->logits_dtype == SJD_BF16  ? launch_pipeline<1>(ra, cfg, smem, grid, stream)
          : P->logits_dtype == SJD_F16 ? launch_pipeline<2>(ra, cfg, smem, grid, stream)
                                       : launch_pipeline<0>(ra, cfg, smem, grid, stream);
    } else {
      const int grid = rows < 4 * sm_count() ? rows : 4 * sm_count();
      e = P->logits_dtype == SJD_BF16
              ? launch_after(sjd::rows_generic_kernel<1, kGenericThreads>, dim3((unsigned)grid), dim3(kGenericThreads), 0, stream, true, ra)
          : P->logits_dtype == SJD_F16
              ? launch_after(sjd::rows_generic_kernel<2, kGenericThreads>, dim3((unsigned)grid), dim3(kGenericThreads), 0, stream, true, ra)
              : launch_after(sjd::rows_generic_kernel<0, kGenericThreads>, dim3((unsigned)grid), dim3(kGenericThreads), 0, stream, true, ra);
    }
    if (e != cudaSuccess) return cuda_fail(e, "row kernel launch");
    ++g_launches;
  }
  if (P->ev_rows_end) {
    const cudaError_t e = cudaEventRecord(static_cast<cudaEvent_t>(P->ev_rows_end), stream);
    if (e != cudaSuccess) return cuda_fail(e, "event record");
  }

  sjd::VerifyArgs va;
  va.B = P->B; va.W = P->W; va.V = P->V; va.kcap = kcap;
  va.flags = P->flags;
  va.tau = P->reuse_tau;
  va.win_len = P->win_len;
  va.pos_base = P->pos_base;
  va.iteration = P->iteration;
  va.iteration0 = P->iteration0;
  va.seq_base = P->seq_base;
  va.seed_lo = ra.seed_lo;
  va.seed_hi = ra.seed_hi;
  va.drafts = drafts;
  va.q_tok = draft_all ? nullptr : draft_probs->tok_prob;
  va.q_ids = draft_all ? nullptr : draft_probs->ids;
  va.q_vals = draft_all ? nullptr : draft_probs->vals;
  va.q_cnt = draft_all ? nullptr : draft_probs->cnt;
  va.p_ids = out_probs->ids;
  va.p_vals = out_probs->vals;
  va.scratch = ra.scratch;
  va.out_accept_len = out_accept_len;
  va.out_tokens = out_tokens;
  va.out_tok_prob = out_probs->tok_prob;
  va.out_flags = P->out_flags;
  va.status = P->status;
  {
    // directly behind the row kernel the verification grid is launched as its programmatic dependent: its
    // blocks are placed as the row kernel's last blocks retire and wait inside the kernel for its completion.
    // An event recorded in between makes it an ordinary launch.
    const cudaError_t e = launch_after(sjd::verify_kernel<kVerifyThreads>, dim3((unsigned)P->B), dim3(kVerifyThreads), 0, stream,
                                       P->ev_rows_end == nullptr, va);
    if (e != cudaSuccess) return cuda_fail(e, "verify kernel launch");
    ++g_launches;
  }
  return SJD_OK;
}

int sjd_step_static(const void* logits_cond, const void* logits_uncond, const int32_t* drafts,
                    const sjd_probs* draft_probs, const sjd_params* P, uint64_t philox_seed, int32_t* out_accept_len,
                    int32_t* out_tokens, sjd_probs* out_probs) {
  if (!P) return SJD_ERR_NULL;
  if (P->struct_size != (int32_t)sizeof(sjd_params)) return SJD_ERR_STRUCT;
  if (P->B < 0 || P->W < 1 || P->W > SJD_W_MAX) return SJD_ERR_SHAPE;
  if ((int64_t)P->B * (int64_t)P->W > (int64_t)SJD_STATIC_MAX_ROWS) return SJD_ERR_CAPACITY;
  void* scratch = nullptr;
  const int rc = static_scratch_address(&scratch);
  if (rc != SJD_OK) return rc;
  sjd_params Q = *P;
  Q.workspace = scratch;
  Q.workspace_bytes = kStaticScratchBytes;
  return sjd_step(logits_cond, logits_uncond, drafts, draft_probs, &Q, philox_seed, out_accept_len, out_tokens, out_probs);
}

}  // extern "C"

namespace {
int fill_advance(sjd::AdvanceArgs* a, const sjd_params* P, int32_t n_total, uint64_t seed, int32_t* win_len,
                 int32_t* pos_base, int32_t* iteration, int32_t* next_drafts, sjd_probs* next_probs) {
  if (!P) return SJD_ERR_NULL;
  if (P->struct_size != (int32_t)sizeof(sjd_params)) return SJD_ERR_STRUCT;
  if (!win_len || !pos_base || !iteration || !next_drafts || check_probs(next_probs) != SJD_OK) return SJD_ERR_NULL;
  if (P->B < 0 || P->W < 1 || P->W > SJD_W_MAX || P->V < 1 || P->top_k < 1 || n_total < 0) return SJD_ERR_SHAPE;
  if (P->init_mode < SJD_INIT_RANDOM || P->init_mode > SJD_INIT_SAMPLE_ABOVE) return SJD_ERR_SHAPE;
  if (P->init_mode != SJD_INIT_RANDOM && P->grid_width < 1) return SJD_ERR_SHAPE;
  std::memset(a, 0, sizeof(*a));
  a->B = P->B; a->W = P->W; a->V = P->V;
  a->kcap = P->top_k < P->V ? P->top_k : P->V;
  a->n_total = n_total;
  a->seq_base = P->seq_base;
  a->init_mode = P->init_mode;
  a->grid_width = P->grid_width > 0 ? P->grid_width : 1;
  a->no_refine = (P->flags & SJD_FLAG_NO_REFINE) ? 1 : 0;
  a->seed_lo = (uint32_t)(seed & 0xffffffffu);
  a->seed_hi = (uint32_t)(seed >> 32);
  a->win_len = win_len; a->pos_base = pos_base; a->iteration = iteration;
  a->next_drafts = next_drafts;
  a->next_tok_prob = next_probs->tok_prob; a->next_ids = next_probs->ids; a->next_vals = next_probs->vals;
  a->next_cnt = next_probs->cnt;
  return SJD_OK;
}
}  // namespace

extern "C" {

int sjd_row_kernel(const sjd_params* P) {
  if (!P) return SJD_ERR_NULL;
  if (P->struct_size != (int32_t)sizeof(sjd_params)) return SJD_ERR_STRUCT;
  if (P->B < 0 || P->W < 1 || P->W > SJD_W_MAX || P->V < 8 || (P->V % 8) != 0 || P->top_k < 1) return SJD_ERR_SHAPE;
  if (P->logits_dtype != SJD_F32 && P->logits_dtype != SJD_BF16 && P->logits_dtype != SJD_F16) return SJD_ERR_DTYPE;
  const int64_t esize = P->logits_dtype == SJD_F32 ? 4 : 2;
  if ((P->stride_b * esize) % 16 != 0 || (P->stride_w * esize) % 16 != 0 || P->stride_w < P->V || P->stride_b < 0)
    return SJD_ERR_ALIGN;
  const int kcap = P->top_k < P->V ? P->top_k : P->V;
  sjd::PipeCfg cfg;
  sjd::RangeCfg rcfg;
  size_t smem = 0;
  const bool fast = !(P->flags & (SJD_FLAG_FORCE_GENERIC | SJD_FLAG_FORCE_TILES));
  if (fast && plan_ranges(P, kcap, &rcfg, &smem, false)) return SJD_ROWS_RANGES;
  if (!(P->flags & SJD_FLAG_FORCE_GENERIC) && plan_pipeline(P, kcap, &cfg, &smem)) return SJD_ROWS_TILES;
  return SJD_ROWS_GENERIC;
}

int sjd_window_init(const sjd_params* P, int32_t n_total, uint64_t philox_seed, int32_t* win_len, int32_t* pos_base,
                    int32_t* iteration, int32_t* drafts, sjd_probs* draft_probs) {
  sjd::AdvanceArgs a;
  const int rc = fill_advance(&a, P, n_total, philox_seed, win_len, pos_base, iteration, drafts, draft_probs);
  if (rc != SJD_OK) return rc;
  if (P->B == 0) return SJD_OK;
  const int rows = P->B * P->W;
  sjd::init_window_kernel<<<(rows + 255) / 256, 256, 0, static_cast<cudaStream_t>(P->stream)>>>(a);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "window init launch");
  ++g_launches;
  return SJD_OK;
}

int sjd_window_advance(const sjd_params* P, int32_t n_total, uint64_t philox_seed, const int32_t* accept_len,
                       const int32_t* step_tokens, const sjd_probs* step_probs, int32_t* win_len, int32_t* pos_base,
                       int32_t* iteration, int32_t* next_drafts, sjd_probs* next_probs, int32_t* committed,
                       int32_t* n_committed) {
  sjd::AdvanceArgs a;
  const int rc = fill_advance(&a, P, n_total, philox_seed, win_len, pos_base, iteration, next_drafts, next_probs);
  if (rc != SJD_OK) return rc;
  if (!accept_len || !step_tokens || !committed || check_probs(const_cast<sjd_probs*>(step_probs)) != SJD_OK) return SJD_ERR_NULL;
  if (P->B == 0) return SJD_OK;
  a.accept_len = accept_len;
  a.step_tokens = step_tokens;
  a.step_tok_prob = step_probs->tok_prob; a.step_ids = step_probs->ids; a.step_vals = step_probs->vals;
  a.step_cnt = step_probs->cnt;
  a.committed = committed;
  a.n_committed = n_committed;
  cudaStream_t st = static_cast<cudaStream_t>(P->stream);
  cudaError_t e = launch_after(sjd::advance_rows_kernel<256>, dim3((unsigned)(P->B * P->W)), dim3(256), 0, st, true, a);
  if (e != cudaSuccess) return cuda_fail(e, "window advance launch");
  ++g_launches;
  e = launch_after(sjd::advance_state_kernel, dim3((unsigned)((P->B + 127) / 128)), dim3(128), 0, st, true, a);
  if (e != cudaSuccess) return cuda_fail(e, "window state launch");
  ++g_launches;
  return SJD_OK;
}

}  // extern "C"

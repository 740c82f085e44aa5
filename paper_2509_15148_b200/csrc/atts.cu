// C-ABI entry points of libatts (declared in include/atts.h): argument checks, launch geometry,
// tensor-map encoding.  All device work is in the kernels of conformal.cuh and lmhead_lse.cuh.
#include "atts.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>
#include <math.h>
#include <stdlib.h>
#include <atomic>
#include <mutex>

#include "conformal.cuh"
#include "lmhead_lse.cuh"

namespace atts {

__device__ unsigned int g_dev_status = 0u;

struct DeviceInfo {
  bool ready = false;                 // the probe has run (under the mutex)
  std::atomic<bool> probed{false};    // set last: a reader that sees it may use every other field without the mutex
  int status = ATTS_OK;  // sticky result of the probe
  int sm_count = 0;
  int pair_workers = 0;  // CTA pairs (clusters of 2) of the fused kernel that can be resident at once; 0 = unusable
  unsigned int* dev_status = nullptr;
  PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
};

static DeviceInfo g_info[64];
static std::mutex g_mu;

// Bound of the scoring kernel's pipeline waits, in SM cycles, and the diagnostic switch that makes the first wait
// run out (atts_debug_set_wait).  The environment variable ATTS_WAIT_LIMIT, read once, presets the bound.
static std::atomic<long long> g_wait_limit{0};   // 0: not set yet
static std::atomic<int> g_withhold_loads{0};
static long long wait_limit() {
  long long v = g_wait_limit.load(std::memory_order_relaxed);
  if (v == 0) {
    v = kWaitLimitCycles;
    if (const char* e = getenv("ATTS_WAIT_LIMIT")) {
      const long long x = atoll(e);
      if (x > 0) v = x;
    }
    g_wait_limit.store(v, std::memory_order_relaxed);
  }
  return v;
}

// Probes the current device once: architecture, SM count, address of the status word, driver entry
// point for tensor-map encoding, and the opt-in shared-memory sizes of the kernels.
static int device_info(const DeviceInfo** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  DeviceInfo& di = g_info[dev];
  if (di.probed.load(std::memory_order_acquire)) {   // every call after the first on a device: no lock
    *out = &di;
    return di.status;
  }
  std::lock_guard<std::mutex> lock(g_mu);
  if (!di.ready) {
    di.ready = true;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
      di.status = ATTS_ERR_CUDA;
    } else if (major != 10) {
      di.status = ATTS_ERR_ARCH;
    } else {
      bool ok = cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess;
      ok = ok && cudaGetSymbolAddress((void**)&di.dev_status, g_dev_status) == cudaSuccess;
      cudaDriverEntryPointQueryResult q;
      void* fn = nullptr;
      ok = ok && cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
           q == cudaDriverEntryPointSuccess && fn != nullptr;
      di.encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
      ok = ok && cudaFuncSetAttribute(lmhead_lse_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      ScoreCfg<1>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(lmhead_lse_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      ScoreCfg<2>::kSmemBytes) == cudaSuccess;
      if (ok) {
        // how many clusters of two CTAs fit the device at once (GPC boundaries may strand an SM)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * (unsigned)di.sm_count);
        cfg.blockDim = dim3(kScoreThreads);
        cfg.dynamicSmemBytes = ScoreCfg<2>::kSmemBytes;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, lmhead_lse_kernel<2>, &cfg) == cudaSuccess && clusters > 0)
          di.pair_workers = clusters < di.sm_count / 2 ? clusters : di.sm_count / 2;
        else
          cudaGetLastError();
      }
      const int rank_smem = 2 * (4 << kRankMaxTableLog2) + 64;  // splitter table + p-value table
      ok = ok && cudaFuncSetAttribute(rank_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, rank_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, rank_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, rank_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, rank_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, rank_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_indexed_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 << kIndexMaxTreeLog2) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_indexed_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 << kIndexMaxTreeLog2) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_indexed_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 << kIndexMaxTreeLog2) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_indexed_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 << kIndexMaxTreeLog2) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_indexed_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 << kIndexMaxTreeLog2) == cudaSuccess;
      const int bucket_smem = 4 * ((1 << kBucketMaxLog2) + 1 + 2 * kBucketMaxN + kBucketPad + 2);
      ok = ok && cudaFuncSetAttribute(rank_bucket_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bucket_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_bucket_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bucket_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_bucket_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bucket_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_bucket_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, bucket_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(rank_bucket_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, bucket_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(small_update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      4 * (kSmallUpdMaxOld + kSmallUpdMaxNew)) == cudaSuccess;
      const int merge_smem = 4 * (2 * kSortMaxK + kMergeTileMax);
      ok = ok && cudaFuncSetAttribute(takeover_ids_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kIdsSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(merge_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, merge_smem) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(merge_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, merge_smem) == cudaSuccess;
      if (!ok) {
        cudaGetLastError();
        di.status = ATTS_ERR_CUDA;
      }
    }
  }
  di.probed.store(true, std::memory_order_release);
  *out = &di;
  return di.status;
}

// Timing hooks: event pairs recorded around the fused kernel while a profiling session is open.
struct Profile {
  bool on = false;
  int cap = 0, used = 0;
  cudaEvent_t* ev = nullptr;  // 2 * cap events
};
static Profile g_prof;

// Launch with the programmatic-serialisation attribute: the kernel may be set up while its predecessor in the
// stream drains; it calls pdl_wait() before it reads anything (see conformal.cuh).
template <typename... KArgs, typename... Args>
static int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) != cudaSuccess) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  return ATTS_OK;
}

static inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
static inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int launch_status() { return cudaGetLastError() == cudaSuccess ? ATTS_OK : ATTS_ERR_CUDA; }

// Workspace layout of atts_score_logprob: [partials C * M_pad float2][gathered M_pad f32][logprob M_pad f32]
struct ScoreWs {
  size_t partial_off, gathered_off, logprob_off, total;
};
static ScoreWs score_ws(const ScorePlan& p) {
  ScoreWs w;
  w.partial_off = 0;
  w.gathered_off = round_up((size_t)p.C * p.M_pad * sizeof(float2), 256);
  w.logprob_off = w.gathered_off + round_up((size_t)p.M_pad * sizeof(float), 256);
  w.total = w.logprob_off + round_up((size_t)p.M_pad * sizeof(float), 256);
  if (w.total == 0) w.total = 256;
  return w;
}

// The schedule of a scoring call.  CTA pairs keep the tensor pipe busier per clock (measured 88-97 % against
// 81-89 %), but once H no longer fits one L2-resident panel their placement (the two CTAs of a cluster and
// neighbouring clusters sit on adjacent SMs) multiplies DRAM traffic and, under the power cap, costs more clock
// than it gains.  So pairs are used when all of H is one panel and their makespan (in tile times) is no longer
// than that of single CTAs; larger batches run on single CTAs.
static ScorePlan choose_score_plan(const DeviceInfo* di, int64_t M, int64_t d, int64_t V) {
  const ScorePlan one = make_score_plan(M, d, V, di->sm_count, 1);
  if (di->pair_workers <= 0 || M == 0) return one;
  const ScorePlan two = make_score_plan(M, d, V, di->pair_workers, 2);
  auto span = [](const ScorePlan& p, int workers) {
    return (long long)((p.units + workers - 1) / workers) * ((p.NT + p.C - 1) / p.C);
  };
  const bool one_panel = two.RB <= two.Gr;
  return (one_panel && span(two, di->pair_workers) <= span(one, di->sm_count)) ? two : one;
}

static int check_score_shape(int64_t M, int64_t d, int64_t V, int64_t S) {
  if (M < 0 || M > (1ll << 30) || S < 0 || S >= (1ll << 31)) return ATTS_ERR_SHAPE;
  if (d < 64 || d > 16384 || d % 64 != 0) return ATTS_ERR_SHAPE;
  if (V < 1 || V >= (1ll << 31) - kBlockN) return ATTS_ERR_SHAPE;
  return ATTS_OK;
}

// A tensor map is a function of the base address, the shape and the box alone, so the last few are kept per host
// thread: a caller that scores batch after batch from the same buffers pays for the encoding once.
struct TmapEntry {
  const void* base = nullptr;
  int64_t rows = 0, cols = 0;
  int box_rows = 0;
  const DeviceInfo* di = nullptr;
  CUtensorMap map;
};
static int encode_2d(const DeviceInfo* di, CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  constexpr int kKept = 8;
  thread_local TmapEntry kept[kKept];
  thread_local int next = 0;
  for (int i = 0; i < kKept; ++i) {
    const TmapEntry& e = kept[i];
    if (e.base == base && e.rows == rows && e.cols == cols && e.box_rows == box_rows && e.di == di) {
      *map = e.map;
      return ATTS_OK;
    }
  }
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = di->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return ATTS_ERR_CUDA;
  TmapEntry& e = kept[next];
  next = (next + 1) % kKept;
  e.base = base; e.rows = rows; e.cols = cols; e.box_rows = box_rows; e.di = di; e.map = *map;
  return ATTS_OK;
}

// Built-in scratch of atts_calib_update_static: the merged copy, ATTS_STATIC_MAX_TOTAL f32.  In host code this name is only a handle for
// cudaGetSymbolAddress; the device address it yields is what kernels are given.
static __device__ __align__(256) unsigned char g_static_scratch[ATTS_STATIC_SCRATCH_BYTES];
static unsigned char* g_static_scratch_addr[64] = {};
static std::mutex g_static_mu;

// Device address of the built-in scratch on the current device, looked up once per device.
static int static_scratch(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return ATTS_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_scratch_addr[dev];
  return ATTS_OK;
}

}  // namespace atts

using namespace atts;

extern "C" {

const char* atts_strerror(int status) {
  switch (status) {
    case ATTS_OK: return "ok";
    case ATTS_ERR_NULL: return "a required pointer is NULL";
    case ATTS_ERR_SHAPE: return "a size is negative, too large or not a supported multiple";
    case ATTS_ERR_ALIGN: return "a pointer is not aligned as required";
    case ATTS_ERR_WORKSPACE: return "the workspace is too small";
    case ATTS_ERR_CAPACITY: return "n + k exceeds the calibration buffer's capacity";
    case ATTS_ERR_ARG: return "a scalar argument is out of range";
    case ATTS_ERR_ARCH: return "the current device is not sm_100 (no fallback path exists)";
    case ATTS_ERR_CUDA: return "a CUDA call failed (no usable device?)";
    case ATTS_ERR_TIMEOUT: return "a bounded wait on the device expired";
    case ATTS_ERR_SCRATCH_LIMIT:
      return "sizes exceed the built-in scratch of the allocation-free entry point (n + k <= 65536, k <= 16384)";
    case ATTS_ERR_INDEX: return "the calibration index was built for another fill of the buffer";
    default: return "unknown status";
  }
}

int atts_version(void) { return 100; }

int atts_score_workspace_bytes(int64_t M, int64_t d, int64_t V, int64_t S, size_t* bytes) {
  if (!bytes) return ATTS_ERR_NULL;
  int st = check_score_shape(M, d, V, S);
  if (st != ATTS_OK) return st;
  const DeviceInfo* di;
  st = device_info(&di);
  if (st != ATTS_OK) return st;
  *bytes = score_ws(choose_score_plan(di, M, d, V)).total;
  return ATTS_OK;
}

// slice_stats != nullptr: W is the vocabulary slice starting at id vocab_offset; the call stops after writing one
// (max, sum, token logit) triple per row (no log-probs, no scores).
static int score_impl(const void* hidden_bf16, const void* lm_head_bf16, const int32_t* token_ids,
                      const float* row_scale, const int32_t* seg_offsets, int64_t M, int64_t d, int64_t V, int64_t S,
                      int32_t score_mode, float* token_logprob, float* sample_score, void* workspace,
                      size_t workspace_bytes, void* cuda_stream, int64_t vocab_offset = 0,
                      float* slice_stats = nullptr) {
  int st = check_score_shape(M, d, V, S);
  if (st != ATTS_OK) return st;
  if (score_mode < 0 || score_mode > 3) return ATTS_ERR_ARG;
  if (!lm_head_bf16 || (!seg_offsets && !slice_stats) || !workspace) return ATTS_ERR_NULL;
  if (M > 0 && (!hidden_bf16 || !token_ids)) return ATTS_ERR_NULL;
  if (S > 0 && !sample_score) return ATTS_ERR_NULL;
  if (!aligned(hidden_bf16, 16) || !aligned(lm_head_bf16, 16) || !aligned(workspace, 256) ||
      !aligned(token_ids, 4) || !aligned(seg_offsets, 4) || !aligned(token_logprob, 4) || !aligned(sample_score, 4) ||
      !aligned(row_scale, 4))
    return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  st = device_info(&di);
  if (st != ATTS_OK) return st;
  ScorePlan plan = choose_score_plan(di, M, d, V);
  plan.vocab_offset = (int)vocab_offset;
  plan.wait_limit = wait_limit();
  plan.withhold_loads = g_withhold_loads.load(std::memory_order_relaxed);
  const ScoreWs ws = score_ws(plan);
  if (workspace_bytes < ws.total) return ATTS_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* wsp = static_cast<uint8_t*>(workspace);
  float2* partial = reinterpret_cast<float2*>(wsp + ws.partial_off);
  float* gathered = reinterpret_cast<float*>(wsp + ws.gathered_off);
  float* logprob_ws = reinterpret_cast<float*>(wsp + ws.logprob_off);

  if (M > 0) {
    CUtensorMap map_h, map_w;
    if (encode_2d(di, &map_h, hidden_bf16, M, d, kBlockM) != ATTS_OK) return ATTS_ERR_CUDA;
    if (encode_2d(di, &map_w, lm_head_bf16, V, d, kBlockN / plan.ctas) != ATTS_OK) return ATTS_ERR_CUDA;
    const bool timed = g_prof.on && g_prof.used < g_prof.cap;
    if (timed) cudaEventRecord(g_prof.ev[2 * g_prof.used], stream);
    if (plan.ctas == 1) {
      const int grid = plan.units < di->sm_count ? plan.units : di->sm_count;
      lmhead_lse_kernel<1><<<grid, kScoreThreads, ScoreCfg<1>::kSmemBytes, stream>>>(map_h, map_w, token_ids, row_scale, plan, partial,
                                                                                     gathered, di->dev_status);
    } else {
      const int pairs = plan.units < di->pair_workers ? plan.units : di->pair_workers;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(2 * (unsigned)pairs);
      cfg.blockDim = dim3(kScoreThreads);
      cfg.dynamicSmemBytes = ScoreCfg<2>::kSmemBytes;
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      if (cudaLaunchKernelEx(&cfg, lmhead_lse_kernel<2>, map_h, map_w, token_ids, row_scale, plan, partial, gathered,
                             di->dev_status) != cudaSuccess) {
        cudaGetLastError();
        return ATTS_ERR_CUDA;
      }
    }
    if (timed) cudaEventRecord(g_prof.ev[2 * g_prof.used++ + 1], stream);
    if ((st = launch_status()) != ATTS_OK) return st;
    if (slice_stats) {
      slice_stats_kernel<<<(unsigned)((M + 255) / 256), 256, 0, stream>>>(partial, gathered, token_ids, (int)M, plan.M_pad,
                                                                          plan.C, (int)V, (int)vocab_offset, slice_stats);
      return launch_status();
    }
    lse_combine_kernel<<<(unsigned)((M + 255) / 256), 256, 0, stream>>>(partial, gathered, token_ids, (int)M, plan.M_pad,
                                                                        plan.C, (int)V, logprob_ws, token_logprob,
                                                                        di->dev_status);
    if ((st = launch_status()) != ATTS_OK) return st;
  }
  if (S > 0) {
    segment_score_kernel<<<(unsigned)S, 256, 0, stream>>>(logprob_ws, seg_offsets, (int)M, (int)S, score_mode, sample_score);
    if ((st = launch_status()) != ATTS_OK) return st;
  }
  return ATTS_OK;
}

int atts_score_logprob(const void* hidden_bf16, const void* lm_head_bf16, const int32_t* token_ids,
                       const int32_t* seg_offsets, int64_t M, int64_t d, int64_t V, int64_t S, int32_t score_mode,
                       float* token_logprob, float* sample_score, void* workspace, size_t workspace_bytes,
                       void* cuda_stream) {
  return score_impl(hidden_bf16, lm_head_bf16, token_ids, nullptr, seg_offsets, M, d, V, S, score_mode, token_logprob,
                    sample_score, workspace, workspace_bytes, cuda_stream);
}

int atts_score_logprob_scaled(const void* hidden_bf16, const void* lm_head_bf16, const int32_t* token_ids,
                              const float* row_scale, const int32_t* seg_offsets, int64_t M, int64_t d, int64_t V,
                              int64_t S, int32_t score_mode, float* token_logprob, float* sample_score, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  if (M > 0 && !row_scale) return ATTS_ERR_NULL;
  return score_impl(hidden_bf16, lm_head_bf16, token_ids, row_scale, seg_offsets, M, d, V, S, score_mode, token_logprob,
                    sample_score, workspace, workspace_bytes, cuda_stream);
}

int atts_score_slice(const void* hidden_bf16, const void* lm_head_slice_bf16, const int32_t* token_ids, int64_t M,
                     int64_t d, int64_t V_slice, int64_t vocab_offset, float* slice_stats, void* workspace,
                     size_t workspace_bytes, void* cuda_stream) {
  if (vocab_offset < 0 || vocab_offset >= (1ll << 31)) return ATTS_ERR_SHAPE;
  if (M > 0 && !slice_stats) return ATTS_ERR_NULL;
  if (!aligned(slice_stats, 4)) return ATTS_ERR_ALIGN;
  if (M == 0) return check_score_shape(M, d, V_slice, 0);
  return score_impl(hidden_bf16, lm_head_slice_bf16, token_ids, nullptr, nullptr, M, d, V_slice, 0, 0, nullptr, nullptr,
                    workspace, workspace_bytes, cuda_stream, vocab_offset, slice_stats);
}

int atts_score_combine(const float* slice_stats, int64_t G, const int32_t* seg_offsets, int64_t M, int64_t S,
                       int32_t score_mode, float* token_logprob, float* sample_score, void* workspace,
                       size_t workspace_bytes, void* cuda_stream) {
  if (M < 0 || M > (1ll << 30) || S < 0 || S >= (1ll << 31) || G < 1 || G > 1024) return ATTS_ERR_SHAPE;
  if (score_mode < 0 || score_mode > 3) return ATTS_ERR_ARG;
  if (!seg_offsets || !workspace || (M > 0 && !slice_stats) || (S > 0 && !sample_score)) return ATTS_ERR_NULL;
  if (!aligned(slice_stats, 4) || !aligned(seg_offsets, 4) || !aligned(token_logprob, 4) || !aligned(sample_score, 4) ||
      !aligned(workspace, 256))
    return ATTS_ERR_ALIGN;
  if (workspace_bytes < round_up((size_t)M * 4, 256) + 256) return ATTS_ERR_WORKSPACE;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  float* logprob_ws = static_cast<float*>(workspace);
  if (M > 0) {
    stats_combine_kernel<<<(unsigned)((M + 255) / 256), 256, 0, stream>>>(slice_stats, (int)G, (int)M, logprob_ws,
                                                                          token_logprob, di->dev_status);
    if ((st = launch_status()) != ATTS_OK) return st;
  }
  if (S > 0) {
    segment_score_kernel<<<(unsigned)S, 256, 0, stream>>>(logprob_ws, seg_offsets, (int)M, (int)S, score_mode, sample_score);
    if ((st = launch_status()) != ATTS_OK) return st;
  }
  return ATTS_OK;
}

int atts_rms_inv(const void* hidden_bf16, int64_t M, int64_t d, float eps, float* row_scale, void* cuda_stream) {
  if (M < 0 || M > (1ll << 30) || d < 8 || d > 16384 || d % 8 != 0) return ATTS_ERR_SHAPE;
  if (!(eps >= 0.f)) return ATTS_ERR_ARG;
  if (M > 0 && (!hidden_bf16 || !row_scale)) return ATTS_ERR_NULL;
  if (!aligned(hidden_bf16, 16) || !aligned(row_scale, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  if (M == 0) return ATTS_OK;
  rms_inv_kernel<<<(unsigned)((M + 7) / 8), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(hidden_bf16), (int)M, (int)d, eps, row_scale);
  return launch_status();
}

// Shared launcher of the rank kernel, with or without the fused thresholding.
static int zero_counts(uint32_t* counts, int n_alpha, cudaStream_t stream) {
  if (counts && cudaMemsetAsync(counts, 0, (size_t)n_alpha * 3 * sizeof(uint32_t), stream) != cudaSuccess) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  return ATTS_OK;
}

// A grid of one block stores its stage counts; larger grids add to counts the host has zeroed.
static int launch_rank(const DeviceInfo* di, const float* scores, int64_t Nc, const float* calib_sorted, int64_t n,
                       uint32_t* numer, float* pvalue, int n_alpha, const FusedClassify& fc, cudaStream_t stream) {
  // Many candidates against a buffer that fits in shared memory: the bucket form (one table lookup and three
  // probes per candidate instead of a log2(n)-step descent).  Its per-block set-up is only repaid by many candidates.
  if (n >= 1 && n <= kBucketMaxN && Nc >= kBucketMinCandidates) {
    int Blog2 = 10;
    while (Blog2 < kBucketMaxLog2 && (1ll << Blog2) < 8 * n) ++Blog2;
    const int64_t per_blk = (int64_t)kRankThreads * kRankPerThread;
    int64_t nblk = (Nc + per_blk - 1) / per_blk;
    if (nblk > di->sm_count) nblk = di->sm_count;
    if (nblk > 1 && n_alpha > 0 && zero_counts(fc.counts, n_alpha, stream) != ATTS_OK) return ATTS_ERR_CUDA;
    const dim3 g((unsigned)nblk), b(kRankThreads);
    const size_t sm = 4 * (((size_t)1 << Blog2) + 1 + (size_t)n + kBucketPad + (pvalue ? (size_t)n + 2 : 0));
    switch (n_alpha) {
      case 0: rank_bucket_kernel<0><<<g, b, sm, stream>>>(scores, Nc, calib_sorted, (int)n, Blog2, numer, pvalue, fc); break;
      case 1: rank_bucket_kernel<1><<<g, b, sm, stream>>>(scores, Nc, calib_sorted, (int)n, Blog2, numer, pvalue, fc); break;
      case 2: rank_bucket_kernel<2><<<g, b, sm, stream>>>(scores, Nc, calib_sorted, (int)n, Blog2, numer, pvalue, fc); break;
      case 3: rank_bucket_kernel<3><<<g, b, sm, stream>>>(scores, Nc, calib_sorted, (int)n, Blog2, numer, pvalue, fc); break;
      default: rank_bucket_kernel<4><<<g, b, sm, stream>>>(scores, Nc, calib_sorted, (int)n, Blog2, numer, pvalue, fc); break;
    }
    return launch_status();
  }
  // Table: the whole buffer when it has at most 8191 entries, else every 2^L-th entry.  Few candidates do
  // not repay a large strided table fill, so they get a smaller one.
  const int64_t max_slots = (Nc >= (1 << 16) ? (1 << kRankMaxTableLog2) : (1 << 10)) - 1;
  int L = 0;
  if (n > (1 << kRankMaxTableLog2) - 1)
    while (((n + (1ll << L) - 1) >> L) > max_slots) ++L;
  const int ns = (int)((n + (1ll << L) - 1) >> L);
  int P = 1;
  while ((1 << P) - 1 < ns) ++P;
  const int64_t per_block = (int64_t)kRankThreads * kRankPerThread;
  int64_t blocks = (Nc + per_block - 1) / per_block;
  // one block per SM when the table is filled by strided loads (the fill is paid per block), two otherwise
  const int64_t max_blocks = (int64_t)di->sm_count * (L == 0 ? 2 : 1);
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks > 1 && n_alpha > 0 && zero_counts(fc.counts, n_alpha, stream) != ATTS_OK) return ATTS_ERR_CUDA;
  const dim3 grid((unsigned)blocks), block(kRankThreads);
  const size_t smem = ((size_t)4 << P) + (L == 0 ? (size_t)4 * (n + 2) : 0);  // table (+ p-value table)
  switch (n_alpha) {
    case 0: rank_kernel<0><<<grid, block, smem, stream>>>(scores, Nc, calib_sorted, (int)n, ns, P, L, numer, pvalue, fc); break;
    case 1: rank_kernel<1><<<grid, block, smem, stream>>>(scores, Nc, calib_sorted, (int)n, ns, P, L, numer, pvalue, fc); break;
    case 2: rank_kernel<2><<<grid, block, smem, stream>>>(scores, Nc, calib_sorted, (int)n, ns, P, L, numer, pvalue, fc); break;
    case 3: rank_kernel<3><<<grid, block, smem, stream>>>(scores, Nc, calib_sorted, (int)n, ns, P, L, numer, pvalue, fc); break;
    default: rank_kernel<4><<<grid, block, smem, stream>>>(scores, Nc, calib_sorted, (int)n, ns, P, L, numer, pvalue, fc); break;
  }
  return launch_status();
}

int atts_conformal_rank(const float* scores, int64_t Nc, const float* calib_sorted, int64_t n, uint32_t* numer,
                        float* pvalue, void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31) || n < 0 || n >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (Nc > 0 && (!scores || !numer)) return ATTS_ERR_NULL;
  if (n > 0 && !calib_sorted) return ATTS_ERR_NULL;
  if (!aligned(scores, 16) || !aligned(numer, 16) || !aligned(pvalue, 16) || !aligned(calib_sorted, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  if (Nc == 0) return ATTS_OK;
  return launch_rank(di, scores, Nc, calib_sorted, n, numer, pvalue, 0, FusedClassify{}, static_cast<cudaStream_t>(cuda_stream));
}

int atts_rank_classify(const float* scores, int64_t Nc, const float* calib_sorted, int64_t n, const double* alphas,
                       int32_t n_alpha, uint32_t* numer, float* pvalue, uint8_t* stage, uint32_t* stage_counts,
                       void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31) || n < 0 || n >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (n_alpha < 1 || n_alpha > kMaxAlphas) return ATTS_ERR_ARG;
  if (!alphas) return ATTS_ERR_NULL;
  for (int a = 0; a < n_alpha; ++a)
    if (!(alphas[a] > 0.0 && alphas[a] < 1.0)) return ATTS_ERR_ARG;
  if (Nc > 0 && (!scores || !numer || !stage)) return ATTS_ERR_NULL;
  if (n > 0 && !calib_sorted) return ATTS_ERR_NULL;
  if (!aligned(scores, 16) || !aligned(numer, 16) || !aligned(pvalue, 16) || !aligned(calib_sorted, 4) ||
      !aligned(stage, 16) || !aligned(stage_counts, 4) || (n_alpha > 1 && Nc % 16 != 0))
    return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (Nc == 0) return zero_counts(stage_counts, n_alpha, stream);
  FusedClassify fc{};
  for (int a = 0; a < n_alpha; ++a) {
    fc.k_alpha[a] = (uint32_t)floor(alphas[a] * (double)(n + 1));
    fc.stage[a] = stage + (size_t)a * Nc;
  }
  fc.counts = stage_counts;
  return launch_rank(di, scores, Nc, calib_sorted, n, numer, pvalue, n_alpha, fc, stream);
}

int atts_classify(const uint32_t* numer, int64_t Nc, int64_t n, double alpha, uint8_t* stage, uint32_t* stage_counts,
                  void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31) || n < 0 || n >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (!(alpha > 0.0 && alpha < 1.0)) return ATTS_ERR_ARG;
  if (Nc > 0 && (!numer || !stage)) return ATTS_ERR_NULL;
  if (!aligned(numer, 16) || !aligned(stage, 16) || !aligned(stage_counts, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (Nc == 0) return zero_counts(stage_counts, 1, stream);
  const uint32_t k_alpha = (uint32_t)floor(alpha * (double)(n + 1));
  const int64_t per_block = (int64_t)kClassifyThreads * kClassifyPerThread;
  int64_t blocks = (Nc + per_block - 1) / per_block;
  const int64_t max_blocks = (int64_t)di->sm_count * 8;
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks > 1 && zero_counts(stage_counts, 1, stream) != ATTS_OK) return ATTS_ERR_CUDA;   // one block stores its counts
  classify_kernel<<<(unsigned)blocks, kClassifyThreads, 0, stream>>>(numer, Nc, k_alpha, stage, stage_counts);
  return launch_status();
}

int atts_threshold(const float* calib_sorted, int64_t n, double alpha, float* tau, void* cuda_stream) {
  if (n < 0 || n >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (!(alpha > 0.0 && alpha < 1.0)) return ATTS_ERR_ARG;
  if (!tau || (n > 0 && !calib_sorted)) return ATTS_ERR_NULL;
  if (!aligned(calib_sorted, 4) || !aligned(tau, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  const int k_alpha = (int)floor(alpha * (double)(n + 1));
  threshold_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(calib_sorted, (int)n, k_alpha, tau);
  return launch_status();
}

int atts_classify_threshold(const float* scores, int64_t Nc, const float* tau, uint8_t* stage, uint32_t* stage_counts,
                            void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31)) return ATTS_ERR_SHAPE;
  if (!tau || (Nc > 0 && (!scores || !stage))) return ATTS_ERR_NULL;
  if (!aligned(scores, 16) || !aligned(stage, 16) || !aligned(stage_counts, 4) || !aligned(tau, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (Nc == 0) return zero_counts(stage_counts, 1, stream);
  const int64_t per_block = (int64_t)kClassifyThreads * kClassifyPerThread;
  int64_t blocks = (Nc + per_block - 1) / per_block;
  const int64_t max_blocks = (int64_t)di->sm_count * 8;
  if (blocks > max_blocks) blocks = max_blocks;
  if (blocks > 1 && zero_counts(stage_counts, 1, stream) != ATTS_OK) return ATTS_ERR_CUDA;   // one block stores its counts
  classify_threshold_kernel<<<(unsigned)blocks, kClassifyThreads, 0, stream>>>(scores, Nc, tau, stage, stage_counts);
  return launch_status();
}

// Workspace of atts_takeover_ids: [one 64-bit word per range][ticket counter], cleared before the launch.  A range
// is at least 8192 stage bytes, which bounds the number of ranges whatever the device.
int atts_takeover_ids_workspace_bytes(int64_t Nc, size_t* bytes) {
  if (!bytes) return ATTS_ERR_NULL;
  if (Nc < 0 || Nc >= (1ll << 31)) return ATTS_ERR_SHAPE;
  *bytes = round_up((size_t)((Nc + 16 + kIdsRowBytes - 1) / kIdsRowBytes) * sizeof(unsigned long long) + 8, 256) + 256;
  return ATTS_OK;
}

int atts_takeover_ids(const uint8_t* stage, int64_t Nc, int32_t* ids, int64_t ids_cap, uint32_t* count, void* workspace,
                      size_t workspace_bytes, void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31) || ids_cap < 0) return ATTS_ERR_SHAPE;
  if ((Nc > 0 && (!stage || !workspace)) || (ids_cap > 0 && !ids)) return ATTS_ERR_NULL;
  if (!aligned(ids, 4) || !aligned(count, 4) || !aligned(workspace, 256)) return ATTS_ERR_ALIGN;
  size_t need = 0;
  atts_takeover_ids_workspace_bytes(Nc, &need);
  if (Nc > 0 && workspace_bytes < need) return ATTS_ERR_WORKSPACE;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (Nc == 0) {
    if (count && cudaMemsetAsync(count, 0, sizeof(uint32_t), stream) != cudaSuccess) {
      cudaGetLastError();
      return ATTS_ERR_CUDA;
    }
    return ATTS_OK;
  }
  // A range is Q rows of 4096 bytes, Q even, 2 <= Q <= 8.  Long ranges even out the lanes' work and cost less per
  // byte, so Q grows as soon as every block that fits the GPU (four per SM) has a range.  The kernel reads whole
  // 16-byte pieces: it starts at the boundary at or below the first stage byte and is told how many bytes to skip.
  const int head = (int)(reinterpret_cast<uintptr_t>(stage) & 15u);
  const uint8_t* base = stage - head;
  const int64_t len = Nc + head;
  const int64_t slots = (int64_t)di->sm_count * 4;
  int64_t Q = (len + kIdsRowBytes * slots - 1) / (kIdsRowBytes * slots);
  Q = (Q + 1) & ~1ll;
  Q = Q < 2 ? 2 : (Q > kIdsMaxRows ? kIdsMaxRows : Q);
  const int ranges = (int)((len + Q * kIdsRowBytes - 1) / (Q * kIdsRowBytes));
  unsigned long long* state = static_cast<unsigned long long*>(workspace);
  unsigned int* ticket = reinterpret_cast<unsigned int*>(state + ranges);
  if (ranges > 1 && cudaMemsetAsync(workspace, 0, (size_t)ranges * sizeof(unsigned long long) + 8, stream) != cudaSuccess) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  const int blocks = ranges < slots ? ranges : (int)slots;
  takeover_ids_kernel<<<blocks, kIdsThreads, kIdsSmemBytes, stream>>>(base, len, head, (int)Q, ranges, state, ticket, ids, ids_cap,
                                                                     count, di->dev_status);
  return launch_status();
}

int atts_conformal_rank_conditional(const float* scores, const int32_t* group_ids, int64_t Nc, const float* calib_segments,
                                    int64_t calib_total, const int32_t* seg_offsets, int64_t G, uint32_t* numer,
                                    uint32_t* denom, float* pvalue, void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31) || G < 0 || G >= (1ll << 31) || calib_total < 0 || calib_total >= (1ll << 31))
    return ATTS_ERR_SHAPE;
  if (Nc > 0 && (!scores || !group_ids || !numer || !denom || !seg_offsets)) return ATTS_ERR_NULL;
  if (Nc > 0 && calib_total > 0 && !calib_segments) return ATTS_ERR_NULL;
  if (!aligned(scores, 4) || !aligned(group_ids, 4) || !aligned(numer, 4) || !aligned(denom, 4) || !aligned(pvalue, 4) ||
      !aligned(calib_segments, 4) || !aligned(seg_offsets, 4))
    return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  if (Nc == 0) return ATTS_OK;
  int64_t blocks = (Nc + 1023) / 1024;
  if (blocks > (int64_t)di->sm_count * 8) blocks = (int64_t)di->sm_count * 8;
  const bool vec4 = aligned(scores, 16) && aligned(group_ids, 16) && aligned(numer, 16) && aligned(denom, 16) &&
                    aligned(pvalue, 16);
  rank_conditional_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      scores, group_ids, Nc, calib_segments, (int)calib_total, seg_offsets, (int)G, numer, denom, pvalue, vec4,
      aligned(calib_segments, 32), di->dev_status);
  return launch_status();
}

int atts_classify_conditional(const uint32_t* numer, const uint32_t* denom, int64_t Nc, double alpha, uint8_t* stage,
                              uint32_t* stage_counts, void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31)) return ATTS_ERR_SHAPE;
  if (!(alpha > 0.0 && alpha < 1.0)) return ATTS_ERR_ARG;
  if (Nc > 0 && (!numer || !denom || !stage)) return ATTS_ERR_NULL;
  if (!aligned(numer, 4) || !aligned(denom, 4) || !aligned(stage_counts, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (stage_counts && cudaMemsetAsync(stage_counts, 0, 3 * sizeof(uint32_t), stream) != cudaSuccess) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  if (Nc == 0) return ATTS_OK;
  int64_t blocks = (Nc + 255) / 256;
  if (blocks > (int64_t)di->sm_count * 8) blocks = (int64_t)di->sm_count * 8;
  classify_conditional_kernel<<<(unsigned)blocks, 256, 0, stream>>>(numer, denom, Nc, alpha, stage, stage_counts);
  return launch_status();
}

// ---- calibration index (see rank_indexed_kernel) ----
static inline size_t index_bytes_for(int64_t cap) { return 4 * index_words((uint32_t)cap); }

// The capacity an index of `index_bytes` bytes is laid out for: the largest one that fits.  Every call that is
// given the same allocation therefore agrees on the layout.
static int64_t index_cap_of_bytes(size_t index_bytes) {
  if (index_bytes < index_bytes_for(0)) return -1;
  int64_t lo = 0, hi = (1ll << 24) - 2;
  while (lo < hi) {
    const int64_t mid = (lo + hi + 1) / 2;
    if (index_bytes_for(mid) <= index_bytes) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Launches the build of slot 0 of the index from src[0, n).
static int launch_index_build(const DeviceInfo* di, const float* src, int64_t n, void* index, int64_t index_cap,
                              cudaStream_t stream) {
  int64_t work = n > 8192 ? n : 8192;
  int64_t blocks = (work + 255) / 256;
  if (blocks > (int64_t)di->sm_count * 8) blocks = (int64_t)di->sm_count * 8;
  index_build_kernel<<<(unsigned)blocks, 256, 0, stream>>>(src, (int)n, (uint32_t)index_cap, static_cast<uint32_t*>(index));
  return launch_status();
}

// Workspace of atts_calib_update: the merged copy, n + k f32.
int atts_calib_workspace_bytes(int64_t n, int64_t k, size_t* bytes) {
  if (!bytes) return ATTS_ERR_NULL;
  if (n < 0 || k < 0 || n + k >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  *bytes = round_up((size_t)(n + k) * 4, 256) + 256;
  return ATTS_OK;
}

// One launch of the merge kernel: kc <= kSortMaxK new scores into cur old entries.  index != nullptr: from the index
// slot of fill `cur` into the other slot and `out` (the caller's buffer); else from calib into `out` (scratch).
static int launch_merge(const DeviceInfo* di, const float* calib, int64_t cur, const float* new_scores, int kc, float* out,
                        void* index, int64_t index_cap, cudaStream_t stream) {
  int k2 = kMergeThreads;   // the block's sort pads its keys to a multiple of the block size
  while (k2 < kc) k2 <<= 1;
  int tile_len = 0, tiles = 0;
  merge_tiling((int)cur, di->sm_count, tile_len, tiles);
  const int blocks = tiles < di->sm_count ? tiles : di->sm_count;
  const size_t smem = (size_t)4 * (2 * (size_t)k2 + (size_t)tile_len);
  if (index)
    return launch_pdl(merge_kernel<true>, dim3(blocks), dim3(kMergeThreads), smem, stream, nullptr, (int)cur, new_scores, kc, k2,
                      tile_len, tiles, out, static_cast<uint32_t*>(index), (uint32_t)index_cap, di->dev_status);
  return launch_pdl(merge_kernel<false>, dim3(blocks), dim3(kMergeThreads), smem, stream, calib, (int)cur, new_scores, kc, k2,
                    tile_len, tiles, out, nullptr, 0u, di->dev_status);
}

static int calib_update_impl(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k, int64_t* n_out,
                             void* workspace, size_t workspace_bytes, void* cuda_stream, void* index, size_t index_bytes) {
  if (n < 0 || k < 0 || cap < 0 || cap >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (n + k > cap) return ATTS_ERR_CAPACITY;
  if ((cap > 0 && !calib) || (k > 0 && (!new_scores || !workspace))) return ATTS_ERR_NULL;
  if (!aligned(calib, 4) || !aligned(new_scores, 4) || !aligned(workspace, 256)) return ATTS_ERR_ALIGN;
  size_t need = 0;
  atts_calib_workspace_bytes(n, k, &need);
  if (k > 0 && workspace_bytes < need) return ATTS_ERR_WORKSPACE;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  int64_t index_cap = 0;
  if (index) {
    if (!aligned(index, 256)) return ATTS_ERR_ALIGN;
    index_cap = index_cap_of_bytes(index_bytes);
    if (index_cap < n + k) return ATTS_ERR_WORKSPACE;
  }
  if (n_out) *n_out = n + k;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (k == 0) return index ? launch_index_build(di, calib, n, index, index_cap, stream) : ATTS_OK;
  // Small problems: one block does it in place in one launch.
  if (n <= kSmallUpdMaxOld && k <= kSmallUpdMaxNew && k * 8 <= n + 64) {
    int k2 = 1;
    while (k2 < k) k2 <<= 1;
    small_update_kernel<<<1, kSmallUpdThreads, (size_t)4 * (k2 + n), stream>>>(calib, (int)n, new_scores, (int)k, k2);
    if ((st = launch_status()) != ATTS_OK) return st;
    return index ? launch_index_build(di, calib, n + k, index, index_cap, stream) : ATTS_OK;
  }
  // One merge launch per slice of at most kSortMaxK new scores: with an index, from one slot of the index into the
  // other and the buffer itself; without, into the workspace followed by a copy back.
  float* merged = static_cast<float*>(workspace);
  int64_t cur = n;
  for (int64_t off = 0; off < k; off += kSortMaxK) {
    const int kc = (int)((k - off) < kSortMaxK ? (k - off) : kSortMaxK);
    const int64_t total = cur + kc;
    if ((st = launch_merge(di, calib, cur, new_scores + off, kc, index ? calib : merged, index, index_cap, stream)) != ATTS_OK)
      return st;
    if (!index && cudaMemcpyAsync(calib, merged, (size_t)total * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
      cudaGetLastError();
      return ATTS_ERR_CUDA;
    }
    cur = total;
  }
  return ATTS_OK;
}

int atts_calib_update(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k, int64_t* n_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return calib_update_impl(calib, n, cap, new_scores, k, n_out, workspace, workspace_bytes, cuda_stream, nullptr, 0);
}

int atts_calib_update_indexed(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k, int64_t* n_out,
                              void* index, size_t index_bytes, void* workspace, size_t workspace_bytes,
                              void* cuda_stream) {
  if (!index) return ATTS_ERR_NULL;
  return calib_update_impl(calib, n, cap, new_scores, k, n_out, workspace, workspace_bytes, cuda_stream, index, index_bytes);
}

int atts_calib_update_static(float* calib, int64_t n, int64_t cap, const float* new_scores, int64_t k, int64_t* n_out,
                             void* cuda_stream) {
  if (n < 0 || k < 0 || cap < 0 || cap >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (n + k > cap) return ATTS_ERR_CAPACITY;
  if (n + k > ATTS_STATIC_MAX_TOTAL || k > ATTS_STATIC_MAX_NEW) return ATTS_ERR_SCRATCH_LIMIT;
  if ((cap > 0 && !calib) || (k > 0 && !new_scores)) return ATTS_ERR_NULL;
  if (!aligned(calib, 4) || !aligned(new_scores, 4)) return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  unsigned char* scratch = nullptr;
  if ((st = static_scratch(&scratch)) != ATTS_OK) return st;
  if (n_out) *n_out = n + k;
  if (k == 0) return ATTS_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  float* merged = reinterpret_cast<float*>(scratch);
  if ((st = launch_merge(di, calib, n, new_scores, (int)k, merged, nullptr, 0, stream)) != ATTS_OK) return st;
  if (cudaMemcpyAsync(calib, merged, (size_t)(n + k) * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  return ATTS_OK;
}

int atts_calib_index_bytes(int64_t cap, size_t* bytes) {
  if (!bytes) return ATTS_ERR_NULL;
  if (cap < 0 || cap >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  *bytes = round_up(index_bytes_for(cap), 256);
  return ATTS_OK;
}

int atts_calib_index_build(const float* calib_sorted, int64_t n, void* index, size_t index_bytes, void* cuda_stream) {
  if (n < 0 || n >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (!index || (n > 0 && !calib_sorted)) return ATTS_ERR_NULL;
  if (!aligned(calib_sorted, 4) || !aligned(index, 256)) return ATTS_ERR_ALIGN;
  const int64_t index_cap = index_cap_of_bytes(index_bytes);
  if (index_cap < n) return ATTS_ERR_WORKSPACE;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  return launch_index_build(di, calib_sorted, n, index, index_cap, static_cast<cudaStream_t>(cuda_stream));
}

int atts_rank_classify_indexed(const float* scores, int64_t Nc, const float* calib_sorted, int64_t n, void* index,
                               const double* alphas, int32_t n_alpha, uint32_t* numer, float* pvalue, uint8_t* stage,
                               uint32_t* stage_counts, void* cuda_stream) {
  if (Nc < 0 || Nc >= (1ll << 31) || n < 0 || n >= (1ll << 24) - 1) return ATTS_ERR_SHAPE;
  if (n_alpha < 0 || n_alpha > kMaxAlphas) return ATTS_ERR_ARG;
  if (n_alpha > 0 && !alphas) return ATTS_ERR_NULL;
  for (int a = 0; a < n_alpha; ++a)
    if (!(alphas[a] > 0.0 && alphas[a] < 1.0)) return ATTS_ERR_ARG;
  if (!index || (Nc > 0 && (!scores || !numer || (n_alpha > 0 && !stage)))) return ATTS_ERR_NULL;
  if (n > 0 && !calib_sorted) return ATTS_ERR_NULL;
  if (!aligned(scores, 16) || !aligned(numer, 16) || !aligned(pvalue, 16) || !aligned(calib_sorted, 4) ||
      !aligned(index, 256) || !aligned(stage, 16) || !aligned(stage_counts, 4) || (n_alpha > 1 && Nc % 16 != 0))
    return ATTS_ERR_ALIGN;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (Nc == 0) return zero_counts(stage_counts, n_alpha, stream);
  FusedClassify fc{};
  for (int a = 0; a < n_alpha; ++a) {
    fc.k_alpha[a] = (uint32_t)floor(alphas[a] * (double)(n + 1));
    fc.stage[a] = stage + (size_t)a * Nc;
  }
  fc.counts = n_alpha > 0 ? stage_counts : nullptr;
  // A buffer that fits in shared memory, or few candidates, gain nothing from the index.
  if (n <= kBucketMaxN || Nc < kIndexMinCandidates)
    return launch_rank(di, scores, Nc, calib_sorted, n, numer, pvalue, n_alpha, fc, stream);
  const IndexShape sh = index_shape(n);
  const int64_t per_block = (int64_t)kRankThreads * kRankPerThread;
  int64_t blocks = (Nc + per_block - 1) / per_block;
  if (blocks > di->sm_count) blocks = di->sm_count;
  const dim3 grid((unsigned)blocks), block(kRankThreads);
  const size_t smem = (size_t)4 << sh.P;
  // The stage counts are gathered in the index header and moved to stage_counts by the last block: no memset node.
  uint32_t* ix = static_cast<uint32_t*>(index);
  switch (n_alpha) {
    case 0: return launch_pdl(rank_indexed_kernel<0>, grid, block, smem, stream, scores, Nc, (int)n, ix, numer, pvalue, fc, di->dev_status);
    case 1: return launch_pdl(rank_indexed_kernel<1>, grid, block, smem, stream, scores, Nc, (int)n, ix, numer, pvalue, fc, di->dev_status);
    case 2: return launch_pdl(rank_indexed_kernel<2>, grid, block, smem, stream, scores, Nc, (int)n, ix, numer, pvalue, fc, di->dev_status);
    case 3: return launch_pdl(rank_indexed_kernel<3>, grid, block, smem, stream, scores, Nc, (int)n, ix, numer, pvalue, fc, di->dev_status);
    default: return launch_pdl(rank_indexed_kernel<4>, grid, block, smem, stream, scores, Nc, (int)n, ix, numer, pvalue, fc, di->dev_status);
  }
}

int atts_last_device_status(void* cuda_stream, uint32_t* bits) {
  if (!bits) return ATTS_ERR_NULL;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned int v = 0;
  if (cudaMemcpyAsync(&v, di->dev_status, sizeof(v), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemsetAsync(di->dev_status, 0, sizeof(v), stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    cudaGetLastError();
    return ATTS_ERR_CUDA;
  }
  *bits = v;
  return (v & ATTS_DEV_WAIT_EXPIRED) ? ATTS_ERR_TIMEOUT : (v & ATTS_DEV_INDEX_STALE) ? ATTS_ERR_INDEX : ATTS_OK;
}

int atts_debug_score_plan(int64_t M, int64_t d, int64_t V, int32_t workers, int32_t ctas, int32_t* out) {
  if (!out) return ATTS_ERR_NULL;
  int st = check_score_shape(M, d, V, 0);
  if (st != ATTS_OK) return st;
  if (workers < 1 || (ctas != 1 && ctas != 2)) return ATTS_ERR_ARG;
  const ScorePlan p = make_score_plan(M, d, V, workers, ctas);
  const int32_t v[8] = {p.RB, p.NT, p.KB, p.C, p.Gr, p.units, p.M_pad, p.ctas};
  for (int i = 0; i < 8; ++i) out[i] = v[i];
  return ATTS_OK;
}

int atts_debug_score_unit(int64_t M, int64_t d, int64_t V, int32_t workers, int32_t ctas, int32_t u, int32_t* out) {
  if (!out) return ATTS_ERR_NULL;
  int st = check_score_shape(M, d, V, 0);
  if (st != ATTS_OK) return st;
  if (workers < 1 || (ctas != 1 && ctas != 2)) return ATTS_ERR_ARG;
  const ScorePlan p = make_score_plan(M, d, V, workers, ctas);
  if (u < 0 || u >= p.units) return ATTS_ERR_ARG;
  int rb, c, nt0, nt1;
  decode_unit(p, u, rb, c, nt0, nt1);
  out[0] = rb; out[1] = c; out[2] = nt0; out[3] = nt1;
  return ATTS_OK;
}

int atts_debug_score_form(int64_t M, int64_t d, int64_t V, int32_t* ctas) {
  if (!ctas) return ATTS_ERR_NULL;
  int st = check_score_shape(M, d, V, 0);
  if (st != ATTS_OK) return st;
  const DeviceInfo* di;
  st = device_info(&di);
  if (st != ATTS_OK) return st;
  *ctas = choose_score_plan(di, M, d, V).ctas;
  return ATTS_OK;
}

int atts_debug_set_wait(int64_t limit_cycles, int32_t withhold_loads) {
  if (withhold_loads != 0 && withhold_loads != 1) return ATTS_ERR_ARG;
  g_wait_limit.store(limit_cycles > 0 ? (long long)limit_cycles : kWaitLimitCycles, std::memory_order_relaxed);
  g_withhold_loads.store(withhold_loads, std::memory_order_relaxed);
  return ATTS_OK;
}

int atts_profile_begin(int max_records) {
  if (max_records < 1 || max_records > 4096) return ATTS_ERR_ARG;
  if (g_prof.on) return ATTS_ERR_ARG;
  const DeviceInfo* di;
  int st = device_info(&di);
  if (st != ATTS_OK) return st;
  g_prof.ev = new cudaEvent_t[2 * max_records];
  for (int i = 0; i < 2 * max_records; ++i) {
    if (cudaEventCreate(&g_prof.ev[i]) != cudaSuccess) {
      for (int j = 0; j < i; ++j) cudaEventDestroy(g_prof.ev[j]);
      delete[] g_prof.ev;
      g_prof.ev = nullptr;
      cudaGetLastError();
      return ATTS_ERR_CUDA;
    }
  }
  g_prof.cap = max_records;
  g_prof.used = 0;
  g_prof.on = true;
  return ATTS_OK;
}

int atts_profile_end(float* ms, int cap, int* count) {
  if (!count || (cap > 0 && !ms)) return ATTS_ERR_NULL;
  if (!g_prof.on) return ATTS_ERR_ARG;
  int st = ATTS_OK;
  for (int i = 0; i < g_prof.used; ++i) {
    float t = 0.f;
    if (cudaEventSynchronize(g_prof.ev[2 * i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&t, g_prof.ev[2 * i], g_prof.ev[2 * i + 1]) != cudaSuccess) {
      cudaGetLastError();
      st = ATTS_ERR_CUDA;
    }
    if (i < cap) ms[i] = t;
  }
  *count = g_prof.used;
  for (int i = 0; i < 2 * g_prof.cap; ++i) cudaEventDestroy(g_prof.ev[i]);
  delete[] g_prof.ev;
  g_prof = Profile{};
  return st;
}

}  // extern "C"

// C ABI of the FLOP hot path (see include/flop.h): argument checks, workspace
// planning, tensor-map creation and kernel launches.  Single translation unit;
// the kernels live in the .cuh files next to it.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <utility>
#include <vector>

#include "../../include/flop.h"
#include "common.cuh"
#include "compact.cuh"
#include "gate_sample.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "gemm_tc_group.cuh"
#include "gemm_tc2_group.cuh"
#include "gemm_tc2_dual.cuh"
#include "gemm_tc2_chain.cuh"
#include "gemm_tc_chainfwd.cuh"
#include "l0_lagrangian.cuh"
#include "wgrad.cuh"
#include "active_ranks.cuh"
#include "gemm_small_t.cuh"
#include "gemm_skinny.cuh"
#include "agp.cuh"
#include "embedding.cuh"

using namespace flop;
typedef __nv_bfloat16 bf16;

namespace {

// FLOP_DEBUG=1 in the environment prints the failing CUDA call to stderr.
inline bool debug_on() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("FLOP_DEBUG"); v = (e && e[0] && e[0] != '0') ? 1 : 0; }
  return v == 1;
}
#define FLOP_CUDA(expr)                                                                           \
  do {                                                                                            \
    cudaError_t e__ = (expr);                                                                     \
    if (e__ != cudaSuccess) {                                                                     \
      if (debug_on()) fprintf(stderr, "[flop] %s:%d: %s -> %s\n", __FILE__, __LINE__, #expr, cudaGetErrorString(e__)); \
      cudaGetLastError();                                                                         \
      return FLOP_ERR_CUDA;                                                                       \
    }                                                                                             \
  } while (0)
#define FLOP_TRY(expr)              \
  do {                              \
    int s__ = (expr);               \
    if (s__ != FLOP_OK) return s__; \
  } while (0)


// Tuning switches.  A library built with -DFLOP_TUNING reads them once from the environment (they exist to
// compare variants on one machine); the normal build takes the defaults below and reads nothing but FLOP_DEBUG.
//   FLOP_NO_PDL=1          launch without programmatic dependent launch
//   FLOP_TC_BN / FLOP_TC_STAGES / FLOP_TC_CTA2 (1 force pairs, 2 forbid)     tile shape of single GEMMs
//   FLOP_TC_GROUP_BN / FLOP_TC_GROUP_CTA2, FLOP_TC_WGRAD_BN / FLOP_TC_WGRAD_CTA2   tile shape of grouped launches
//   FLOP_NO_TMA_STORE=1    bf16 output tiles by per-thread stores    FLOP_NO_SCHED=1   round-robin tile order
//   FLOP_NO_SMALL_T=1, FLOP_NO_SKINNY=1   few-token forward kernels off
//   FLOP_STAGE_MERGE=0     backward in three launches per stage instead of two shared ones
//   FLOP_GATHER_PIPE=0     plain P gather kernel                     FLOP_NO_CHAIN=1   chained calls run unchained
//   FLOP_CHAIN_STAGES=2    chained calls put dependent products in ONE launch (default 1: a launch per stage)
//   FLOP_SCHED_EPI=c       per-tile fixed cost (SM cycles) in the tile schedule's cost model instead of 400 + 4 bn
struct Tuning {
  int no_pdl = 0, tc_bn = 0, tc_stages = 0, tc_cta2 = 0, no_tma_store = 0, no_sched = 0, group_bn = 0, group_cta2 = 0,
      wgrad_bn = 0, wgrad_cta2 = 0, no_small_t = 0, no_skinny = 0, stage_merge = 1, gather_pipe = 1, no_chain = 0, chain_stages = 1, sched_epi = 0;
};
inline const Tuning& tuning() {
  static const Tuning t = [] {
    Tuning v;
#ifdef FLOP_TUNING
    auto get = [](const char* name, int dflt) { const char* e = getenv(name); return e ? atoi(e) : dflt; };
    v.no_pdl = get("FLOP_NO_PDL", 0); v.tc_bn = get("FLOP_TC_BN", 0); v.tc_stages = get("FLOP_TC_STAGES", 0);
    v.tc_cta2 = get("FLOP_TC_CTA2", 0); v.no_tma_store = get("FLOP_NO_TMA_STORE", 0); v.no_sched = get("FLOP_NO_SCHED", 0);
    v.group_bn = get("FLOP_TC_GROUP_BN", 0); v.group_cta2 = get("FLOP_TC_GROUP_CTA2", 0); v.wgrad_bn = get("FLOP_TC_WGRAD_BN", 0);
    v.wgrad_cta2 = get("FLOP_TC_WGRAD_CTA2", 0); v.no_small_t = get("FLOP_NO_SMALL_T", 0); v.no_skinny = get("FLOP_NO_SKINNY", 0);
    v.stage_merge = get("FLOP_STAGE_MERGE", 1); v.gather_pipe = get("FLOP_GATHER_PIPE", 1); v.no_chain = get("FLOP_NO_CHAIN", 0);
    v.chain_stages = get("FLOP_CHAIN_STAGES", 1); v.sched_epi = get("FLOP_SCHED_EPI", 0);
#endif
    return v;
  }();
  return t;
}

// Every kernel goes through here: programmatic dependent launch lets a kernel's prologue overlap
// the tail of its predecessor on the stream (the kernels call griddepcontrol.wait before they
// touch global memory).
inline bool pdl_on() { return !tuning().no_pdl; }
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_on() ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);   // errors are picked up by cudaGetLastError()
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline bool valid_dt(int dt) { return dt == FLOP_F32 || dt == FLOP_BF16; }
inline size_t elt(int dt) { return dt == FLOP_BF16 ? 2 : 4; }
inline bool valid_hc(const flop_hc_params_t& hc) { return hc.beta > 0.f && hc.gamma < 0.f && hc.zeta > 1.f; }

// Per-device state (function attributes already set, SM count, built-in scratch address) is indexed by the
// current device, so that a process that drives several GPUs configures each of them.
constexpr int kMaxDevices = 64;
inline int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
  return (dev >= 0 && dev < kMaxDevices) ? dev : -1;
}
// True the first time it is called for (flag array, current device): the caller then sets its function attributes.
inline bool first_use_on_device(bool (&done)[kMaxDevices]) {
  const int dev = current_device();
  if (dev < 0) return true;            // unknown device: configure every time
  if (done[dev]) return false;
  done[dev] = true;
  return true;
}

int num_sms() {
  static int cached[kMaxDevices] = {};
  const int dev = current_device();
  if (dev >= 0 && cached[dev]) return cached[dev];
  int n = 0;
  if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return 148;   // B200; used only for planning when no device is visible
  }
  cached[dev] = n;
  return n;
}


// ------------------------------------------------------------------ instrumentation
// Host-side count of kernels launched by this library, and optional CUDA-event timing of
// the tensor-core GEMM launches (flop_gemm_timing_begin/end): events are recorded on the
// launching stream around every tensor-core GEMM launch and summed when timing ends.
unsigned long long g_launches = 0;
struct GemmTiming {
  bool on = false;
  std::vector<cudaEvent_t> ev;   // pairs (start, stop)
  size_t used = 0;
  double flops = 0.0;
} g_timing;
std::mutex g_timing_mu;

inline void count_launch(int n = 1) { g_launches += (unsigned long long)n; }

// Device-side stamps (flop_gemm_stamps_begin/end): while on, GEMM launch i writes its start and end
// %globaltimer to stamps[2i], stamps[2i+1] of a caller-provided device buffer.
struct GemmStamps {
  unsigned long long* buf = nullptr;
  int capacity = 0, used = 0;
  double flops = 0.0;
} g_stamps;

struct GemmTimer {
  cudaStream_t st;
  bool active;
  cudaEvent_t stop = nullptr;
  GemmTimer(cudaStream_t s, double flops) : st(s), active(false) {
    if (!g_timing.on) return;
    std::lock_guard<std::mutex> lk(g_timing_mu);
    if (g_timing.used + 2 > g_timing.ev.size()) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        g_timing.ev.push_back(e);
      }
    }
    cudaEventRecord(g_timing.ev[g_timing.used], st);
    stop = g_timing.ev[g_timing.used + 1];
    g_timing.used += 2;
    g_timing.flops += flops;
    active = true;
  }
  ~GemmTimer() { if (active) cudaEventRecord(stop, st); }
};

// ------------------------------------------------------------------ bump allocator over ws
struct Arena {
  unsigned char* base;
  size_t size, used;
  void* take(size_t bytes) {
    const size_t off = align_up(used, 256);
    used = off + bytes;
    return base ? base + off : nullptr;
  }
};

// ------------------------------------------------------------------ tensor-core GEMM planning
struct TcPlan {
  int bn, stages, tiles_m, tiles_n, splits, kb_per_split, num_kb;
  int cta2;   // 1: pairs of CTAs compute 256 x bn tiles (gemm2_group_kernel); 0: one CTA per 128 x bn tile
};

constexpr int kSmemBudget = 227 * 1024 - 1024;   // opt-in maximum minus room for the static __shared__ variables
constexpr int kSmemBarrierBytes = 384;   // pipeline barriers (8 x (2 x 8 + 5) bytes) and the chained kernel's queue ring (160 bytes)
constexpr int kSmemFixed = 1024 + (int)tc::kStoreBufTotal + kSmemBarrierBytes;   // alignment slack + epilogue staging + barriers


// Picks the tile shape (one CTA: 128 x bn; CTA pair: 256 x bn), and the split-K factor, by a small
// cost model in SM cycles: waves over the machine x (k-blocks per work item x the slower of MMA
// issue and shared-memory fill, plus the epilogue).  The fill rate of one SM's shared memory was
// measured at about 54 bytes per cycle; a 128 x bn x 64 MMA block takes 2*bn cycles.
TcPlan plan_tc(int64_t M, int64_t N, int64_t K, bool allow_split, bool b_mn_major, bool allow_cta2 = true) {
  const int sms = num_sms();
  const int num_kb = (int)((K + tc::BK - 1) / tc::BK);
  const int force_bn = tuning().tc_bn, force_stages = tuning().tc_stages, force_cta2 = tuning().tc_cta2;
  TcPlan best{};
  double best_cost = 1e300;
  // 208 (two tiles cover a 410-wide matrix; CTA pairs, K-major B) is offered only when asked for: at Transformer-XL
  // sizes it removes a fifth of the tensor-core work of the forward products and changes nothing (4.28 against
  // 4.26 ms per step: those tiles are bound by their stores, not by the MMAs)
  const int bns[5] = {256, 208, 192, 128, 64};
  for (int pass = 0; pass < 2 && best_cost == 1e300; ++pass)   // second pass: overrides that fit no tile are dropped
  for (int cta2 = 0; cta2 <= 1; ++cta2) {
    if (cta2 && !allow_cta2) continue;
    if (pass == 0 && allow_cta2 && ((force_cta2 == 1 && !cta2) || (force_cta2 == 2 && cta2))) continue;
    for (int bi = 0; bi < 5; ++bi) {
      const int bn = bns[bi];
      if (bn == 208 && (force_bn != 208 || !cta2 || b_mn_major)) continue;
      const bool forced_bn = pass == 0 && force_bn;
      if (forced_bn && bn != force_bn) continue;
      if (!forced_bn && bn > 64 && bn - 64 >= N) continue;   // a smaller tile already covers N
      if (cta2 && b_mn_major && (bn / 2) % 64 != 0) continue;  // MN-major halves come in 64-wide boxes
      const int bm = cta2 ? tc::BM2 : tc::BM;
      const int units = cta2 ? sms / 2 : sms;                 // CTA pairs or CTAs that run at once
      const int tiles_m = (int)((M + bm - 1) / bm), tiles_n = (int)((N + bn - 1) / bn);
      const int max_split = allow_split ? std::min(num_kb, 32) : 1;
      const double bytes = cta2 ? (double)tc::stage_bytes2(bn) : (double)tc::stage_bytes(bn);
      for (int sp = 1; sp <= max_split; ++sp) {
        const int kbps = (num_kb + sp - 1) / sp;
        const int splits = (num_kb + kbps - 1) / kbps;
        if (splits != sp) continue;
        const double items = (double)tiles_m * tiles_n * splits;
        const double waves = ceil(items / units);
        const double per_kb = std::max(2.0 * bn, bytes / 54.0);
        const double epi = 600.0 + 10.0 * bn;
        double cost = waves * (kbps * per_kb + epi) + 3000.0;
        if (splits > 1) cost += 0.004 * (double)splits * (double)M * (double)N / sms;   // ordered reduction pass
        if (cost < best_cost) {
          best_cost = cost;
          best.bn = bn; best.tiles_m = tiles_m; best.tiles_n = tiles_n; best.cta2 = cta2;
          best.splits = splits; best.kb_per_split = kbps; best.num_kb = num_kb;
        }
      }
    }
  }
  const int sb = best.cta2 ? (int)tc::stage_bytes2(best.bn) : (int)tc::stage_bytes(best.bn);
  best.stages = std::min(tc::kMaxStages, (kSmemBudget - 1024 - kSmemBarrierBytes) / sb);
  if (force_stages > 0) best.stages = std::min(best.stages, force_stages);
  return best;
}

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  });
  return fn;
}

// Row-major bf16 matrix [rows, cols] with leading dimension ld; box = box_cols x box_rows, 128-byte swizzle.
int make_tmap(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    if (debug_on()) fprintf(stderr, "[flop] cuTensorMapEncodeTiled entry point not found\n");
    return FLOP_ERR_CUDA;
  }
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS && debug_on())
    fprintf(stderr, "[flop] cuTensorMapEncodeTiled failed (%d): ptr=%p rows=%lld cols=%lld ld=%lld box=%ux%u\n", (int)r, ptr,
            (long long)rows, (long long)cols, (long long)ld, box_cols, box_rows);
  return r == CUDA_SUCCESS ? FLOP_OK : FLOP_ERR_CUDA;
}

// Operand of D = sum_k A(m,k) B(n,k) taken from a row-major matrix.
struct Operand {
  const void* ptr;
  int64_t ld;
  bool mn_major;   // false: memory is [MN rows, K cols]; true: memory is [K rows, MN cols]
};

struct TcEpilogue {
  int kind;   // tc::EPI_STORE or tc::EPI_SLICE
  bf16* out; int64_t ldo; const float* col_scale;
  float* slices; int64_t slice_elems, ld_slice;
  const bf16* qdot; int64_t ldq; float* dz_part; int64_t dz_stride; int* dz_meta;
  void* wg_out; int wg_f32; const float* row_scale; int accumulate;   // tc::EPI_WGRAD (ldo is shared with out)
};

TcEpilogue store_epilogue(void* out, int64_t ldo, const float* col_scale) {
  TcEpilogue e{};
  e.kind = tc::EPI_STORE; e.out = (bf16*)out; e.ldo = ldo; e.col_scale = col_scale;
  return e;
}

// ---- grouped launches: several independent GEMMs of the same kind in one persistent kernel
struct TcJob {
  Operand A, B;
  int64_t M, N, K;
  TcPlan pl;
  TcEpilogue ep;
  const int* dyn_m = nullptr;   // effective sizes on the device (see tc::Params), nullable
  const int* dyn_n = nullptr;
  const int* dyn_k = nullptr;
  // chained launches (gemm_tc2_chain.cuh): stage 0 waits for nothing, stage 1 reads a stage-0 output; inside a
  // stage a unit walks lower classes first; link holds the counters and the folded-in side work
  int stage = 0, order_class = 0;
  tc::ChainLink link{};
};

template <bool A_MN, bool B_MN, int EPI>
int launch_group_inst(const tc::GroupParams& gp, int cta2, double flops, cudaStream_t st) {
  static bool configured[kMaxDevices] = {};
  auto kern1 = tc::gemm_group_kernel<A_MN, B_MN, EPI>;
  auto kern2 = tc::gemm2_group_kernel<A_MN, B_MN, EPI>;
  if (first_use_on_device(configured)) {
    FLOP_CUDA(cudaFuncSetAttribute(kern1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
    FLOP_CUDA(cudaFuncSetAttribute(kern2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
  }
  {
    GemmTimer timer(st, flops);
    if (!cta2) {
      const int smem = kSmemFixed + gp.stages * (int)tc::stage_bytes(gp.bn_max);
      launch_k(kern1, dim3(gp.sched.n_units ? gp.sched.n_units : std::min(gp.total_work, num_sms())), dim3(tc::kThreads), (size_t)smem, st, gp);
    } else {
      const int smem = kSmemFixed + gp.stages * (int)tc::stage_bytes2(gp.bn_max);
      const int pairs = gp.sched.n_units ? gp.sched.n_units : std::min(gp.total_work, num_sms() / 2);
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(tc::kThreads); cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = st;
      cudaLaunchAttribute attr[2];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[1].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = pdl_on() ? 2 : 1;
      cudaLaunchKernelEx(&cfg, kern2, gp);
    }
  }
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

// A launch whose problems are of two kinds: bf16 stores with (K-major A, MN-major B) and in-place weight
// gradients with both operands MN-major (the two steps of the grouped backward pass).  CTA pairs only.
int launch_dual_inst(const tc::GroupParams& gp, double flops, cudaStream_t st) {
  static bool configured[kMaxDevices] = {};
  auto kern = tc::gemm2_dual_kernel<false, true, tc::EPI_STORE, true, true, tc::EPI_WGRAD>;
  if (first_use_on_device(configured)) FLOP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
  {
    GemmTimer timer(st, flops);
    const int smem = kSmemFixed + gp.stages * (int)tc::stage_bytes2(gp.bn_max);
    const int pairs = gp.sched.n_units ? gp.sched.n_units : std::min(gp.total_work, num_sms() / 2);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(tc::kThreads); cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_on() ? 2 : 1;
    cudaLaunchKernelEx(&cfg, kern, gp);
  }
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

// Fills the next problem slot of a launch from a job: tensor maps, sizes, epilogue, work-list position; appends
// the cost of each of its work items (SM cycles, the model of plan_group) for the schedule.
int add_problem(tc::GroupParams& gp, const TcJob& j, std::vector<double>& item_cost, double& flops) {
  if (j.M > INT32_MAX || j.N > INT32_MAX || j.K > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  const bool kind1 = j.A.mn_major && j.B.mn_major && j.ep.kind == tc::EPI_WGRAD;
  tc::GroupProblem& pr = gp.prob[gp.n];
  pr.p.kind = kind1 ? 1 : 0;
  if (!j.A.mn_major) FLOP_TRY(make_tmap(&pr.ta, j.A.ptr, j.M, j.K, j.A.ld, tc::BK, tc::BM));
  else               FLOP_TRY(make_tmap(&pr.ta, j.A.ptr, j.K, j.M, j.A.ld, tc::kBoxMN, tc::BK));
  if (!j.B.mn_major) FLOP_TRY(make_tmap(&pr.tb, j.B.ptr, j.N, j.K, j.B.ld, tc::BK, (uint32_t)(j.pl.cta2 ? j.pl.bn / 2 : j.pl.bn)));
  else               FLOP_TRY(make_tmap(&pr.tb, j.B.ptr, j.K, j.N, j.B.ld, tc::kBoxMN, tc::BK));
  tc::Params& p = pr.p;
  p.M = (int)j.M; p.N = (int)j.N; p.K = (int)j.K;
  p.bn = j.pl.bn; p.stages = 0; p.tiles_m = j.pl.tiles_m; p.tiles_n = j.pl.tiles_n;
  p.splits = j.pl.splits; p.kb_per_split = j.pl.kb_per_split; p.num_kb = j.pl.num_kb;
  {
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n, items = tiles * std::max(p.splits, 1);
    p.div_fast = items < 65536 ? 1 : 0;
    p.magic_tn = p.tiles_n > 1 ? (uint32_t)(0x100000000ull / (uint64_t)p.tiles_n) + 1u : 0u;
    p.magic_tiles = (p.div_fast && tiles > 1) ? (uint32_t)(0x100000000ull / (uint64_t)tiles) + 1u : 0u;
  }
  p.out = j.ep.out; p.ldo = j.ep.ldo; p.col_scale = j.ep.col_scale;
  p.slices = j.ep.slices; p.slice_elems = j.ep.slice_elems; p.ld_slice = j.ep.ld_slice;
  p.qdot = j.ep.qdot; p.ldq = j.ep.ldq; p.dz_part = j.ep.dz_part; p.dz_stride = j.ep.dz_stride; p.dz_meta = j.ep.dz_meta;
  p.wg_out = j.ep.wg_out; p.wg_f32 = j.ep.wg_f32; p.row_scale = j.ep.row_scale; p.accumulate = j.ep.accumulate;
  p.dyn_m = j.dyn_m; p.dyn_n = j.dyn_n; p.dyn_k = j.dyn_k;
  p.link = j.link;
  // bf16 tiles that are plainly overwritten leave through a TMA store (64 x 32 boxes of the output)
  void* tma_dst = j.ep.kind == tc::EPI_STORE ? (void*)j.ep.out
                  : (j.ep.kind == tc::EPI_WGRAD && !j.ep.wg_f32 && !j.ep.accumulate) ? j.ep.wg_out : nullptr;
  p.tma_store = (tma_dst && !tuning().no_tma_store) ? 1 : 0;
  if (p.tma_store) FLOP_TRY(make_tmap(&pr.tout, tma_dst, j.M, j.N, j.ep.ldo, 64, 32));
  pr.work_begin = gp.total_work;
  gp.total_work += p.tiles_m * p.tiles_n * p.splits;
  const double bytes = j.pl.cta2 ? (double)tc::stage_bytes2(p.bn) : (double)tc::stage_bytes(p.bn);
  const double per_kb = std::max(2.0 * p.bn, bytes / 50.0), epi = tuning().sched_epi > 0 ? (double)tuning().sched_epi : 400.0 + 4.0 * p.bn;
  if (item_cost.size() <= (size_t)tc::kMaxSched)
    for (int sp = 0; sp < p.splits; ++sp) {
      const int kbs = std::min(p.kb_per_split, p.num_kb - sp * p.kb_per_split);
      item_cost.insert(item_cost.end(), (size_t)p.tiles_m * p.tiles_n, kbs * per_kb + epi);
    }
  gp.bn_max = std::max(gp.bn_max, p.bn);
  flops += 2.0 * j.M * (double)j.N * j.K;
  ++gp.n;
  return FLOP_OK;
}

inline void attach_stamp(tc::GroupParams& gp, double flops) {
  gp.stamp = nullptr;
  if (g_stamps.buf && g_stamps.used < g_stamps.capacity) {
    gp.stamp = g_stamps.buf + 2 * g_stamps.used++;
    g_stamps.flops += flops;
  }
}

int launch_tc_group(const std::vector<TcJob>& jobs, cudaStream_t st) {
  size_t i = 0;
  while (i < jobs.size()) {
    tc::GroupParams gp;
    memset(&gp, 0, sizeof(gp));
    double flops = 0.0;
    const TcJob& first = jobs[i];
    bool uniform = true, dual_ok = true;   // one kind of problem / the two kinds gemm2_dual_kernel is built for
    std::vector<double> item_cost;
    for (; i < jobs.size() && gp.n < tc::kMaxGroup; ++i) {
      const TcJob& j = jobs[i];
      if (j.M <= 0 || j.N <= 0 || j.K <= 0) continue;
      if (j.pl.cta2 != first.pl.cta2) return FLOP_ERR_INVALID_ARG;
      if (j.A.mn_major != first.A.mn_major || j.B.mn_major != first.B.mn_major || j.ep.kind != first.ep.kind) uniform = false;
      const bool kind0 = !j.A.mn_major && j.B.mn_major && j.ep.kind == tc::EPI_STORE;
      const bool kind1 = j.A.mn_major && j.B.mn_major && j.ep.kind == tc::EPI_WGRAD;
      if (!(kind0 || kind1) || !j.pl.cta2) dual_ok = false;
      FLOP_TRY(add_problem(gp, j, item_cost, flops));
    }
    if (gp.n == 0) continue;
    const int cta2 = first.pl.cta2;
    gp.stages = std::min(tc::kMaxStages, (kSmemBudget - kSmemFixed) /
                                             (int)(cta2 ? tc::stage_bytes2(gp.bn_max) : tc::stage_bytes(gp.bn_max)));
    attach_stamp(gp, flops);
    // Tiles of unequal length: deal them out by the longest-processing-time rule when that beats the
    // round-robin order.
    {
      const int units = std::min(gp.total_work, cta2 ? num_sms() / 2 : num_sms());
      double rr = 0.0;
      if (tuning().no_sched || (int)item_cost.size() != gp.total_work) {
        gp.sched.n_units = 0;
      } else {
        const double lpt = tc::build_schedule(item_cost, units, &gp.sched, &rr);
        if (lpt < 0.0 || lpt > 0.97 * rr) gp.sched.n_units = 0;
        if (gp.sched.n_units) {     // every entry also names its problem, so that no role has to search for it
          static_assert(tc::kMaxSched <= (1 << tc::kSchedProblemShift) && tc::kMaxGroup <= (1 << (16 - tc::kSchedProblemShift)), "entry bits");
          for (int i = 0; i < gp.total_work; ++i) {
            const int w = gp.sched.item[i];
            int g = 0;
            for (int k = 1; k < gp.n; ++k)
              if (w >= gp.prob[k].work_begin) g = k;
            gp.sched.item[i] = (uint16_t)((g << tc::kSchedProblemShift) | w);
          }
        }
      }
    }
    const bool a_mn = first.A.mn_major, b_mn = first.B.mn_major;
    int rc = FLOP_ERR_UNSUPPORTED;
    if (!uniform) rc = dual_ok ? launch_dual_inst(gp, flops, st) : FLOP_ERR_INVALID_ARG;
    else if (!a_mn && !b_mn && first.ep.kind == tc::EPI_STORE) rc = launch_group_inst<false, false, tc::EPI_STORE>(gp, cta2, flops, st);
    else if (!a_mn && b_mn && first.ep.kind == tc::EPI_STORE) rc = launch_group_inst<false, true, tc::EPI_STORE>(gp, cta2, flops, st);
    else if (a_mn && b_mn && first.ep.kind == tc::EPI_SLICE) rc = launch_group_inst<true, true, tc::EPI_SLICE>(gp, cta2, flops, st);
    else if (a_mn && b_mn && first.ep.kind == tc::EPI_WGRAD) rc = launch_group_inst<true, true, tc::EPI_WGRAD>(gp, cta2, flops, st);
    FLOP_TRY(rc);
  }
  return FLOP_OK;
}

// ---- chained launch: the tiles of two dependent GEMM stages in ONE persistent CTA-pair launch (gemm_tc2_chain.cuh)
constexpr size_t kSyncBytes = 64 * 1024;   // size of a sync area (flop_sync_bytes)

template <bool A0, bool B0, int E0, bool A1, bool B1, int E1>
int launch_chain_inst(const tc::GroupParams& gp, int pairs, double flops, cudaStream_t st) {
  static bool configured[kMaxDevices] = {};
  auto kern = tc::gemm2_chain_kernel<A0, B0, E0, A1, B1, E1>;
  if (first_use_on_device(configured)) FLOP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
  {
    GemmTimer timer(st, flops);
    const int smem = kSmemFixed + gp.stages * (int)tc::stage_bytes2(gp.bn_max);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(tc::kChainThreads); cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_on() ? 2 : 1;
    cudaLaunchKernelEx(&cfg, kern, gp);
  }
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

// Whether a set of jobs can run as one chained launch: CTA-pair tiles throughout, no split-K, at most
// kMaxGroup problems, and a sync area that holds `sync_words` counters.
bool chain_ok(const std::vector<TcJob>& jobs, const void* sync, size_t sync_bytes, size_t sync_words) {
  if (!sync || tuning().no_chain || jobs.empty() || jobs.size() > (size_t)tc::kMaxGroup) return false;
  if (sync_words * 4 > std::min(sync_bytes, kSyncBytes)) return false;
  for (const TcJob& j : jobs)
    if (!j.pl.cta2 || j.pl.splits != 1 || j.M <= 0 || j.N <= 0 || j.K <= 0) return false;
  return true;
}

// jobs: stage-0 jobs first (when the queue table cannot hold the launch the kernel walks the work list in order).
// backward = the two kinds of the backward pass (bf16 store with MN-major B / in-place weight gradient), else bf16
// stores with both operands K-major.  dep_job[i] = index of the job whose output job i reads (-1: none).
int launch_tc_chain(const std::vector<TcJob>& jobs, const std::vector<int>& dep_job, unsigned* sync, int sync_words, bool backward,
                    cudaStream_t st) {
  tc::GroupParams gp;
  memset(&gp, 0, sizeof(gp));
  double flops = 0.0;
  std::vector<double> item_cost;
  struct Item { int job, tm; };
  std::vector<Item> items;
  bool side = false;
  for (size_t i = 0; i < jobs.size(); ++i) {
    const TcJob& j = jobs[i];
    if (i > 0 && j.stage < jobs[i - 1].stage) return FLOP_ERR_INVALID_ARG;
    FLOP_TRY(add_problem(gp, j, item_cost, flops));
    for (int tm = 0; tm < j.pl.tiles_m; ++tm)
      for (int tn = 0; tn < j.pl.tiles_n; ++tn) items.push_back(Item{(int)i, tm});
    if (j.link.sw_qz) side = true;
  }
  gp.stages = std::min(tc::kMaxStages, (kSmemBudget - kSmemFixed) / (int)tc::stage_bytes2(gp.bn_max));
  attach_stamp(gp, flops);
  const int pairs = std::max(1, std::min(gp.total_work, num_sms() / 2));
  // Queue order.  First stage: by class (tiles that others wait for first), long tiles before short ones, then by
  // row block and problem.  Second stage: by class, then in the order in which the tiles they wait for leave the
  // queue, long before short.
  gp.sched.n_units = 0;
  const int n = (int)items.size();
  if ((int)item_cost.size() == n && n == gp.total_work && n <= tc::kMaxSched) {
    const int64_t kCostMax = (int64_t)1 << 30;
    auto inv_cost = [&](int i) { return kCostMax - std::min<int64_t>(kCostMax - 1, (int64_t)item_cost[(size_t)i]); };
    std::vector<int> stage((size_t)n);
    std::vector<int64_t> key((size_t)n, 0);
    std::vector<int> first;   // stage-0 items
    for (int i = 0; i < n; ++i) {
      const TcJob& j = jobs[(size_t)items[(size_t)i].job];
      stage[(size_t)i] = j.stage;
      if (j.stage == 0) {
        key[(size_t)i] = ((int64_t)j.order_class << 60) | (inv_cost(i) << 28) | ((int64_t)items[(size_t)i].tm << 8) | (int64_t)items[(size_t)i].job;
        first.push_back(i);
      }
    }
    std::stable_sort(first.begin(), first.end(), [&](int a, int b) { return key[(size_t)a] < key[(size_t)b]; });
    // position in the queue at which the last tile of (job, row block) is drawn, and of the whole job
    std::vector<std::vector<int>> ready(jobs.size());
    std::vector<int> ready_all(jobs.size(), 0);
    for (size_t q = 0; q < jobs.size(); ++q) ready[q].assign((size_t)std::max(1, jobs[q].pl.tiles_m), 0);
    for (size_t pos = 0; pos < first.size(); ++pos) {
      const Item& it = items[(size_t)first[pos]];
      ready[(size_t)it.job][(size_t)it.tm] = (int)pos;
      ready_all[(size_t)it.job] = (int)pos;
    }
    for (int i = 0; i < n; ++i) {
      const Item& it = items[(size_t)i];
      const TcJob& j = jobs[(size_t)it.job];
      if (j.stage == 0) continue;
      const int d = dep_job[(size_t)it.job];
      int r = 0;
      if (d >= 0) r = j.link.dep_mode == 1 ? ready[(size_t)d][(size_t)std::min<int>(it.tm, (int)ready[(size_t)d].size() - 1)] : ready_all[(size_t)d];
      key[(size_t)i] = ((int64_t)j.order_class << 60) | ((int64_t)r << 40) | (inv_cost(i) << 8) | (int64_t)it.job;
    }
    tc::build_chain_queue(stage, key, &gp.sched);
  }
  gp.sync = sync;
  gp.sync_words = sync_words;
  gp.side_need = side ? (unsigned)(2 * pairs * tc::kSideWarps) : 0u;
  if (backward) return launch_chain_inst<false, true, tc::EPI_STORE, true, true, tc::EPI_WGRAD>(gp, pairs, flops, st);
  return launch_chain_inst<false, false, tc::EPI_STORE, false, false, tc::EPI_STORE>(gp, pairs, flops, st);
}


// A single GEMM is a group of one.
int launch_tc(const Operand& A, const Operand& B, int64_t M, int64_t N, int64_t K, const TcPlan& pl,
              const TcEpilogue& ep, cudaStream_t st) {
  TcJob j{A, B, M, N, K, pl, ep};
  return launch_tc_group(std::vector<TcJob>{j}, st);
}

// ---- tile shape for a whole group: one (pair?, N tile) for all jobs of a launch, no split-K
TcPlan fixed_plan(int64_t M, int64_t N, int64_t K, int bn, int cta2) {
  TcPlan pl{};
  const int bm = cta2 ? tc::BM2 : tc::BM;
  pl.bn = bn; pl.cta2 = cta2; pl.splits = 1;
  pl.tiles_m = (int)((M + bm - 1) / bm); pl.tiles_n = (int)((N + bn - 1) / bn);
  pl.num_kb = (int)((K + tc::BK - 1) / tc::BK); pl.kb_per_split = pl.num_kb;
  return pl;
}
struct Mnk { int64_t M, N, K; };
struct GroupShape { int bn, cta2; double items; };
// Cost in SM cycles of running all jobs with one tile shape: rounds over the machine x (average
// k-blocks per tile x the slower of MMA issue and shared-memory fill) + epilogues.  The fill rate
// of an SM (about 50 B/clk) is what usually decides, which favours CTA pairs and wide tiles;
// padding waste and the number of rounds pull the other way.
GroupShape plan_group(const std::vector<Mnk>& jobs, bool b_mn_major, bool wgrad = false, bool pairs_only = false) {
  const int force_bn_all = tuning().group_bn, force_cta2_all = tuning().group_cta2;
  const int force_bn_w = tuning().wgrad_bn, force_cta2_w = tuning().wgrad_cta2;
  const int force_bn = wgrad && force_bn_w ? force_bn_w : force_bn_all;
  const int force_cta2 = wgrad && force_cta2_w ? force_cta2_w : force_cta2_all;
  const int sms = num_sms();
  GroupShape best{0, 0, 0.0};
  double best_cost = 1e300;
  const int cand[5] = {256, 208, 192, 128, 64};
  for (int pass = 0; pass < 2 && best.bn == 0; ++pass)
  for (int cta2 = 0; cta2 <= 1; ++cta2) {
    if (pass == 0 && ((force_cta2 == 1 && !cta2) || (force_cta2 == 2 && cta2))) continue;
    if (pairs_only && !cta2) continue;
    for (int c = 0; c < 5; ++c) {
      const int bn = cand[c];
      if (bn == 208 && (force_bn != 208 || !cta2 || b_mn_major)) continue;
      if (pass == 0 && force_bn && bn != force_bn) continue;
      if (cta2 && b_mn_major && (bn / 2) % 64 != 0) continue;
      const int bm = cta2 ? tc::BM2 : tc::BM;
      const int units = cta2 ? sms / 2 : sms;
      double items = 0, kb_sum = 0;
      for (const Mnk& j : jobs) {
        const double t = (double)((j.M + bm - 1) / bm) * (double)((j.N + bn - 1) / bn);
        items += t;
        kb_sum += t * (double)((j.K + tc::BK - 1) / tc::BK);
      }
      if (items <= 0) continue;
      const double bytes = cta2 ? (double)tc::stage_bytes2(bn) : (double)tc::stage_bytes(bn);
      const double per_kb = std::max(2.0 * bn, bytes / 50.0);
      const double rounds = ceil(items / units);
      const double cost = rounds * ((kb_sum / items) * per_kb + 400.0 + 4.0 * bn) + 3000.0;
      if (cost < best_cost) { best_cost = cost; best = GroupShape{bn, cta2, items}; }
    }
  }
  return best;
}

// Weight gradient written straight from the GEMM epilogue (no split-K, no fp32 slices).
TcEpilogue wgrad_epilogue(void* out, int64_t ldo, int wgrad_dt, const float* row_scale, int accumulate) {
  TcEpilogue e{};
  e.kind = tc::EPI_WGRAD; e.wg_out = out; e.ldo = ldo; e.wg_f32 = wgrad_dt == FLOP_F32; e.row_scale = row_scale; e.accumulate = accumulate;
  return e;
}
// The direct epilogue stores 16-byte vectors: rows of the output must allow that.
bool wgrad_direct_ok(const void* out, int64_t ldo, int wgrad_dt) {
  return aligned16(out) && (ldo % (wgrad_dt == FLOP_F32 ? 4 : 8)) == 0;
}

// On-chip forward chain (gemm_tc_chainfwd.cuh): Y = ((X Q^T) * z) P^T in one launch, H' kept in shared memory.
// FLOP_ERR_UNSUPPORTED when the rank does not fit (k > 512) -- the caller then runs the two products as two launches.
int launch_chain_fwd(const void* X, int64_t ldx, const void* Q, int64_t ldq, const void* P, int64_t ldp, const float* z, void* Y,
                     int64_t ldy, int64_t T, int64_t d_in, int64_t d_out, int64_t k, cudaStream_t st) {
  if (k < 1 || k > tc::kChainMaxK || T < 1 || d_in < 1 || d_out < 1 || T > INT32_MAX || d_in > INT32_MAX || d_out > INT32_MAX)
    return FLOP_ERR_UNSUPPORTED;
  const int64_t row_blocks = (T + tc::BM - 1) / tc::BM;
  if (row_blocks > 65535) return FLOP_ERR_UNSUPPORTED;
  static bool configured[kMaxDevices] = {};
  if (first_use_on_device(configured))
    FLOP_CUDA(cudaFuncSetAttribute(tc::chain_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc::kChainSmemBytes));
  tc::ChainFwdParams cp;
  memset(&cp, 0, sizeof(cp));
  FLOP_TRY(make_tmap(&cp.tx, X, T, d_in, ldx, tc::BK, tc::BM));
  FLOP_TRY(make_tmap(&cp.tq, Q, k, d_in, ldq, tc::BK, 64));
  FLOP_TRY(make_tmap(&cp.tp, P, d_out, k, ldp, tc::BK, tc::kChainBN));
  FLOP_TRY(make_tmap(&cp.ty, Y, T, d_out, ldy, 64, 32));
  cp.z = z;
  cp.T = (int)T; cp.d_in = (int)d_in; cp.d_out = (int)d_out; cp.k = (int)k; cp.k_pad = (int)round_up(k, 64);
  cp.tiles_n = (int)((d_out + tc::kChainBN - 1) / tc::kChainBN);
  // Every CTA of a row block recomputes H, so a row block is cut into as few slices as fill the machine.
  const int slices = (int)std::min<int64_t>(cp.tiles_n, std::max<int64_t>(1, num_sms() / row_blocks));
  cp.tiles_per_cta = (cp.tiles_n + slices - 1) / slices;
  tc::Params& y = cp.y;
  y.M = (int)T; y.N = (int)d_out; y.K = (int)k; y.bn = tc::kChainBN; y.tiles_n = cp.tiles_n; y.tiles_m = (int)row_blocks;
  y.splits = 1; y.out = (bf16*)Y; y.ldo = ldy; y.tma_store = 1;
  const dim3 grid((unsigned)((cp.tiles_n + cp.tiles_per_cta - 1) / cp.tiles_per_cta), (unsigned)row_blocks);
  {
    GemmTimer timer(st, 2.0 * (double)T * (double)k * ((double)d_in + (double)d_out));
    launch_k(tc::chain_fwd_kernel, grid, dim3(tc::kThreads), (size_t)tc::kChainSmemBytes, st, cp);
  }
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

// Few-token forward product C = (A B^T) * col_scale on the CUDA cores (see gemm_small_t.cuh).
// Returns FLOP_ERR_UNSUPPORTED when the shape does not fit (the caller then uses the tensor-core path).
template <int TT>
int launch_small_t_inst(const bf16* A, int64_t lda, const bf16* B, int64_t ldb, bf16* C, int64_t ldc, const float* cs, int T,
                        int N, int K, int k_pad, size_t smem, cudaStream_t st) {
  static bool configured[kMaxDevices] = {};
  if (first_use_on_device(configured)) FLOP_CUDA(cudaFuncSetAttribute(small_t_gemm_kernel<TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
  const int grid = std::min((N + kSmallTWarps - 1) / kSmallTWarps, num_sms() * 4);
  launch_k(small_t_gemm_kernel<TT>, dim3(grid), dim3(32 * kSmallTWarps), smem, st, A, lda, B, ldb, C, ldc, cs, T, N, K, k_pad);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}
int launch_small_t(const void* A, int64_t lda, const void* B, int64_t ldb, void* C, int64_t ldc, const float* cs, int64_t T,
                   int64_t N, int64_t K, cudaStream_t st) {
  const int off = tuning().no_small_t;
  if (off || T < 1 || T > kSmallTMax || N > INT32_MAX || K > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  int tt = 1;
  while (tt < T) tt *= 2;
  const int k_pad = (int)round_up(K, 256);                 // every lane's 8-element step stays inside the row
  const size_t smem = (size_t)tt * k_pad * 2;
  if (smem > (size_t)kSmemBudget) return FLOP_ERR_UNSUPPORTED;
  const bf16* a = (const bf16*)A; const bf16* b = (const bf16*)B; bf16* c = (bf16*)C;
  switch (tt) {
    case 1: return launch_small_t_inst<1>(a, lda, b, ldb, c, ldc, cs, (int)T, (int)N, (int)K, k_pad, smem, st);
    case 2: return launch_small_t_inst<2>(a, lda, b, ldb, c, ldc, cs, (int)T, (int)N, (int)K, k_pad, smem, st);
    default: return launch_small_t_inst<4>(a, lda, b, ldb, c, ldc, cs, (int)T, (int)N, (int)K, k_pad, smem, st);
  }
}

// Forward product for 5..16 tokens with warp-level tensor-core instructions (see gemm_skinny.cuh).
template <int MT>
int launch_skinny_inst(const bf16* A, int64_t lda, const bf16* B, int64_t ldb, bf16* C, int64_t ldc, const float* cs, int T, int N,
                       int K, int k_pad, size_t smem, cudaStream_t st) {
  static bool configured[kMaxDevices] = {};
  if (first_use_on_device(configured)) FLOP_CUDA(cudaFuncSetAttribute(skinny_gemm_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget));
  const int groups = (N + 7) / 8;
  const int grid = std::min((groups + kSkinnyWarps - 1) / kSkinnyWarps, num_sms() * 2);
  launch_k(skinny_gemm_kernel<MT>, dim3(grid), dim3(32 * kSkinnyWarps), smem, st, A, lda, B, ldb, C, ldc, cs, T, N, K, k_pad);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}
int launch_skinny(const void* A, int64_t lda, const void* B, int64_t ldb, void* C, int64_t ldc, const float* cs, int64_t T, int64_t N,
                  int64_t K, cudaStream_t st) {
  const int off = tuning().no_skinny;
  if (off || T < 1 || T > kSkinnyMaxT || N > INT32_MAX || K > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  const int mt = (int)((T + 15) / 16);
  const int k_pad = (int)round_up(K, 32);
  const size_t smem = (size_t)16 * mt * (k_pad + kSkinnyPad) * 2;
  if (smem > (size_t)kSmemBudget) return FLOP_ERR_UNSUPPORTED;
  const bf16* a = (const bf16*)A; const bf16* b = (const bf16*)B; bf16* c = (bf16*)C;
  switch (mt) {
    case 1: return launch_skinny_inst<1>(a, lda, b, ldb, c, ldc, cs, (int)T, (int)N, (int)K, k_pad, smem, st);
    default: return FLOP_ERR_UNSUPPORTED;
  }
}
// Few-token forward: CUDA-core streaming up to 4 tokens, warp-level tensor cores up to 16.
int launch_few_tokens(const void* A, int64_t lda, const void* B, int64_t ldb, void* C, int64_t ldc, const float* cs, int64_t T,
                      int64_t N, int64_t K, cudaStream_t st) {
  if (T <= kSmallTMax) return launch_small_t(A, lda, B, ldb, C, ldc, cs, T, N, K, st);
  return launch_skinny(A, lda, B, ldb, C, ldc, cs, T, N, K, st);
}

int launch_simt(const float* A, int64_t a_sm, int64_t a_sk, const float* B, int64_t b_sn, int64_t b_sk, float* C,
                int64_t ldc, int64_t M, int64_t N, int64_t K, const float* col_scale, const float* row_scale,
                int accumulate, cudaStream_t st) {
  if (M <= 0 || N <= 0) return FLOP_OK;
  if (M > INT32_MAX || N > INT32_MAX || K > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  SimtGemmArgs a{A, a_sm, a_sk, B, b_sn, b_sk, C, ldc, (int)M, (int)N, (int)K, col_scale, row_scale, accumulate};
  const dim3 grid((unsigned)((N + 63) / 64), (unsigned)((M + 63) / 64));
  if (grid.y > 65535) return FLOP_ERR_UNSUPPORTED;
  launch_k(simt_gemm_kernel, dim3(grid), dim3(256), (size_t)(0), st, a);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

template <typename T>
int zero_2d(void* out, int64_t ld, int64_t rows, int64_t cols, cudaStream_t st) {
  if (!out || rows <= 0 || cols <= 0) return FLOP_OK;
  const int64_t n = rows * cols;
  launch_k(fill_zero_2d_kernel<T>, dim3((unsigned)((n + 255) / 256)), dim3(256), (size_t)(0), st, (T*)out, ld, (int)rows, (int)cols);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

bool check_mat(const void* p, int64_t ld, int64_t cols) { return p != nullptr && ld >= cols; }
bool bf16_ok(const void* p, int64_t ld) { return aligned16(p) && (ld % 8) == 0; }

// Workspace layouts (shared by the size query and the calls).
struct FwdWs { void* H; int64_t ldh; size_t bytes; };
FwdWs plan_fwd_ws(Arena& ar, int64_t T, int64_t r, int dt) {
  FwdWs w{};
  w.ldh = round_up(std::max<int64_t>(r, 1), 8);
  w.H = ar.take((size_t)T * w.ldh * elt(dt));
  w.bytes = ar.used;
  return w;
}

struct BwdWs {
  void* dH; int64_t lddh;        // dH'[T, r]
  void* Qz; int64_t ldqz;        // diag(z) Q [r, d_in]
  float* slices_p; float* slices_q;   // fp32 split-K slices of dY^T H' and dH'^T X
  int64_t ld_slice_p, ld_slice_q, slice_elems_p, slice_elems_q;
  float* dz_part; int n_part;
  int* dz_meta;                  // device word: partial vectors the last backward call left in dz_part
  TcPlan plan_p, plan_q;
  size_t bytes;
};
BwdWs plan_bwd_ws(Arena& ar, int64_t T, int64_t d_in, int64_t d_out, int64_t r, int dt, bool grouped = false) {
  BwdWs w{};
  w.lddh = round_up(std::max<int64_t>(r, 1), 8);
  w.dH = ar.take((size_t)T * w.lddh * elt(dt));
  w.ldqz = round_up(std::max<int64_t>(d_in, 1), 8);
  w.Qz = ar.take((size_t)r * w.ldqz * elt(dt));
  w.ld_slice_p = round_up(std::max<int64_t>(r, 1), 4);
  w.ld_slice_q = round_up(std::max<int64_t>(d_in, 1), 4);
  int sp = 1, sq = 1;
  w.n_part = 1;
  if (dt == FLOP_BF16) {
    w.plan_p = plan_tc(d_out, r, T, true, true, !grouped);
    w.plan_q = plan_tc(r, d_in, T, true, true, !grouped);
    sp = std::max(1, w.plan_p.splits);
    sq = std::max(1, w.plan_q.splits);
    w.n_part = 2 * sq * std::max(1, w.plan_q.tiles_n);   // per split, N tile and epilogue-warp half
  }
  w.slice_elems_p = d_out * w.ld_slice_p;
  w.slice_elems_q = r * w.ld_slice_q;
  w.slices_p = dt == FLOP_BF16 ? (float*)ar.take((size_t)sp * w.slice_elems_p * 4) : nullptr;
  w.slices_q = (float*)ar.take((size_t)sq * w.slice_elems_q * 4);
  // room for the partials of any tile shape: the direct-epilogue path may use another N tile than plan_q
  const int64_t part_cap = std::max<int64_t>(w.n_part, 2 * ((d_in + 63) / 64));
  w.dz_part = (float*)ar.take((size_t)part_cap * std::max<int64_t>(r, 1) * 4);
  w.dz_meta = (int*)ar.take(256);
  w.bytes = ar.used;
  return w;
}

size_t l0_ws_bytes(int64_t n, int64_t n_seg) {
  const int64_t chunks = (n + kL0Chunk - 1) / kL0Chunk + n_seg;
  return sizeof(L0Scratch) + (size_t)std::max<int64_t>(chunks, 1) * sizeof(double);
}

int check_ws(const void* ws, size_t ws_bytes, size_t need) {
  if (need == 0) return FLOP_OK;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0 || ws_bytes < need) return FLOP_ERR_WORKSPACE;
  return FLOP_OK;
}


// ------------------------------------------------------------------ built-in scratch (no-allocation entry point)
// Scratch of flop_expected_l0_lagrangian_noalloc: a fixed device array that is part of the
// loaded library image (every GPU that loads the library holds it until the process exits).
// Sized for kNoAllocMaxGates gates in kNoAllocMaxSeg segments.
constexpr int64_t kNoAllocMaxGates = 1 << 20;
constexpr int kNoAllocMaxSeg = kL0MaxSeg;
constexpr size_t kNoAllocScratchBytes =
    sizeof(L0Scratch) + (size_t)(kNoAllocMaxGates / kL0Chunk + kNoAllocMaxSeg) * sizeof(double);
static __device__ __align__(256) unsigned char g_l0_builtin_scratch[kNoAllocScratchBytes];

// In host code the array's name is only a handle; the device address comes from the runtime,
// asked once per device with that device current.
void* g_l0_builtin_ptr[kMaxDevices] = {};
std::mutex g_l0_builtin_mu;

int builtin_scratch(L0Scratch** out) {
  int dev = -1;
  FLOP_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return FLOP_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lk(g_l0_builtin_mu);
  if (!g_l0_builtin_ptr[dev]) {
    void* p = nullptr;
    FLOP_CUDA(cudaGetSymbolAddress(&p, g_l0_builtin_scratch));
    if (!p) return FLOP_ERR_CUDA;
    g_l0_builtin_ptr[dev] = p;
  }
  *out = reinterpret_cast<L0Scratch*>(g_l0_builtin_ptr[dev]);
  return FLOP_OK;
}

}  // namespace

template <typename TW, typename TQ>
static int finalize_wgrad(const float* slices, int n_slices, int64_t slice_elems, int64_t ld_slice, int64_t M, int64_t N,
                          const float* row_scale, void* out, int64_t ldo, int accumulate, const void* qdot, int64_t ldq,
                          float* dz_out, cudaStream_t st) {
  if (M <= 0) return FLOP_OK;
  launch_k(wgrad_finalize_kernel<TW, TQ>, dim3((unsigned)M), dim3(256), (size_t)(0), st, slices, n_slices, slice_elems, ld_slice, (int)M, (int)N, row_scale,
                                                            (TW*)out, ldo, accumulate, (const TQ*)qdot, ldq, dz_out);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

// ====================================================================== C ABI
extern "C" {

const char* flop_status_string(int status) {
  switch (status) {
    case FLOP_OK: return "ok";
    case FLOP_ERR_INVALID_ARG: return "invalid argument";
    case FLOP_ERR_UNSUPPORTED: return "unsupported shape, alignment or size";
    case FLOP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FLOP_ERR_CUDA: return "CUDA call failed";
    case FLOP_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int flop_last_async_status(void* stream) {
  FLOP_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  int v = 0;
  FLOP_CUDA(cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)));
  if (v != 0) {
    const int zero = 0;
    FLOP_CUDA(cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)));
  }
  return v;
}

int flop_device_status(void* stream) { return flop_last_async_status(stream); }

int flop_selftest_wait_timeout(int64_t limit_cycles, int* gave_up_dev, void* stream) {
  if (limit_cycles <= 0 || limit_cycles > 2000000000LL || !gave_up_dev) return FLOP_ERR_INVALID_ARG;
  launch_k(tc::wait_selftest_kernel, dim3(1), dim3(32), (size_t)0, (cudaStream_t)stream, (long long)limit_cycles, gave_up_dev);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

unsigned long long flop_launch_count(void) { return g_launches; }

int flop_plan_tile_schedule(const double* cost, int32_t n, int32_t units, int32_t* unit_of_item, double* makespan,
                            double* rr_makespan) {
  if (n < 0 || (n > 0 && !cost) || n > tc::kMaxSched || units < 1 || units > tc::kMaxUnits) return FLOP_ERR_INVALID_ARG;
  std::vector<double> c(cost, cost + n);
  static tc::Schedule sched;   // 4 KB: kept off the stack
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  double rr = 0.0;
  const double ms = tc::build_schedule(c, units, &sched, &rr);
  const bool table = sched.n_units > 0;   // otherwise the launch keeps the round-robin deal (it is within 3 % of the bound)
  if (makespan) *makespan = n > 0 ? (table ? ms : rr) : 0.0;
  if (rr_makespan) *rr_makespan = rr;
  if (unit_of_item && n > 0) {
    if (table) {
      for (int u = 0; u < units; ++u)
        for (int i = sched.begin[u]; i < sched.begin[u + 1]; ++i) unit_of_item[sched.item[i]] = u;
    } else {
      for (int i = 0; i < n; ++i) unit_of_item[i] = i % units;
    }
  }
  return FLOP_OK;
}

int flop_plan_chain_queue(const int32_t* stage, const int64_t* key, int32_t n, int32_t* queue_pos) {
  if (n < 0 || (n > 0 && (!stage || !key)) || n > tc::kMaxSched) return FLOP_ERR_INVALID_ARG;
  if (n == 0) return FLOP_OK;
  static tc::Schedule sched;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  if (!tc::build_chain_queue(std::vector<int>(stage, stage + n), std::vector<int64_t>(key, key + n), &sched)) return FLOP_ERR_INVALID_ARG;
  if (queue_pos)
    for (int i = 0; i < n; ++i) queue_pos[sched.item[i]] = i;
  return FLOP_OK;
}

int flop_gemm_stamps_begin(unsigned long long* stamps_dev, int capacity) {
  if (!stamps_dev || capacity <= 0) return FLOP_ERR_INVALID_ARG;
  g_stamps.buf = stamps_dev; g_stamps.capacity = capacity; g_stamps.used = 0; g_stamps.flops = 0.0;
  return FLOP_OK;
}

// acc[0] += sum over the stamp pairs of (end - start) where both were written; acc[1] += 1.
__global__ void __launch_bounds__(256)
stamps_accumulate_kernel(const unsigned long long* __restrict__ stamps, int capacity, unsigned long long* __restrict__ acc) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ unsigned long long part[8];
  unsigned long long s = 0;
  for (int i = threadIdx.x; i < capacity; i += blockDim.x) {
    const unsigned long long a = stamps[2 * i], e = stamps[2 * i + 1];
    if (a != 0 && e > a) s += e - a;
  }
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int w = 0; w < 8; ++w) t += part[w];
    acc[0] += t;
    acc[1] += 1;
  }
}

int flop_gemm_stamps_accumulate(const unsigned long long* stamps_dev, int capacity, unsigned long long* acc_dev, void* stream) {
  if (!stamps_dev || capacity <= 0 || !acc_dev) return FLOP_ERR_INVALID_ARG;
  launch_k(stamps_accumulate_kernel, dim3(1), dim3(256), (size_t)0, (cudaStream_t)stream, stamps_dev, capacity, acc_dev);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

int flop_gemm_stamps_end(int* launches, double* total_flops) {
  if (launches) *launches = g_stamps.used;
  if (total_flops) *total_flops = g_stamps.flops;
  g_stamps.buf = nullptr; g_stamps.capacity = 0;
  return FLOP_OK;
}

int flop_gemm_timing_begin(void) {
  std::lock_guard<std::mutex> lk(g_timing_mu);
  g_timing.used = 0;
  g_timing.flops = 0.0;
  g_timing.on = true;
  return FLOP_OK;
}

int flop_gemm_timing_end(double* total_ms, double* total_flops, int64_t* launches) {
  std::lock_guard<std::mutex> lk(g_timing_mu);
  g_timing.on = false;
  double ms = 0.0;
  for (size_t i = 0; i + 1 < g_timing.used; i += 2) {
    FLOP_CUDA(cudaEventSynchronize(g_timing.ev[i + 1]));
    float t = 0.f;
    FLOP_CUDA(cudaEventElapsedTime(&t, g_timing.ev[i], g_timing.ev[i + 1]));
    ms += (double)t;
  }
  if (total_ms) *total_ms = ms;
  if (total_flops) *total_flops = g_timing.flops;
  if (launches) *launches = (int64_t)(g_timing.used / 2);
  return FLOP_OK;
}

int flop_tc_gemm(const void* A, int64_t lda, int a_mn_major, const void* B, int64_t ldb, int b_mn_major, void* D,
                 int64_t ldd, const float* col_scale, float* slices, int64_t M, int64_t N, int64_t K, int bn, int cta2,
                 int splits, int* n_slices_out, void* stream) {
  if (M < 0 || N < 0 || K < 0 || !A || !B) return FLOP_ERR_INVALID_ARG;
  if (!bf16_ok(A, lda) || !bf16_ok(B, ldb)) return FLOP_ERR_UNSUPPORTED;
  const bool slice = a_mn_major && b_mn_major;
  if (a_mn_major && !b_mn_major) return FLOP_ERR_UNSUPPORTED;
  if (slice ? (slices == nullptr) : (D == nullptr || !bf16_ok(D, ldd) || ldd < N)) return FLOP_ERR_INVALID_ARG;
  TcPlan pl = plan_tc(M, N, K, slice, b_mn_major != 0);
  if (bn > 0 || cta2 >= 0 || splits > 0) {   // explicit tile shape
    if (bn > 0) pl.bn = bn;
    if (cta2 >= 0) pl.cta2 = cta2;
    if (pl.bn != 64 && pl.bn != 128 && pl.bn != 192 && pl.bn != 208 && pl.bn != 256) return FLOP_ERR_INVALID_ARG;
    if (pl.bn == 208 && (!pl.cta2 || b_mn_major)) return FLOP_ERR_UNSUPPORTED;
    if (pl.cta2 && b_mn_major && (pl.bn / 2) % 64 != 0) return FLOP_ERR_UNSUPPORTED;
    const int bm = pl.cta2 ? tc::BM2 : tc::BM;
    pl.tiles_m = (int)((M + bm - 1) / bm);
    pl.tiles_n = (int)((N + pl.bn - 1) / pl.bn);
    pl.num_kb = (int)((K + tc::BK - 1) / tc::BK);
    int sp = splits > 0 ? splits : pl.splits;
    if (!slice) sp = 1;
    sp = std::max(1, std::min(sp, std::max(pl.num_kb, 1)));
    pl.kb_per_split = (pl.num_kb + sp - 1) / sp;
    pl.splits = pl.kb_per_split > 0 ? (pl.num_kb + pl.kb_per_split - 1) / pl.kb_per_split : 1;
    const int sb = pl.cta2 ? (int)tc::stage_bytes2(pl.bn) : (int)tc::stage_bytes(pl.bn);
    pl.stages = std::min(tc::kMaxStages, (kSmemBudget - 1024 - kSmemBarrierBytes) / sb);
  }
  TcEpilogue e{};
  if (slice) {
    e.kind = tc::EPI_SLICE; e.slices = slices; e.ld_slice = round_up(std::max<int64_t>(N, 1), 4); e.slice_elems = M * e.ld_slice;
  } else {
    e = store_epilogue(D, ldd, col_scale);
  }
  FLOP_TRY(launch_tc({A, lda, a_mn_major != 0}, {B, ldb, b_mn_major != 0}, M, N, K, pl, e, (cudaStream_t)stream));
  if (n_slices_out) *n_slices_out = pl.splits;
  return FLOP_OK;
}

static size_t embedding_ws_bytes(int64_t T, int64_t d_i);

int flop_workspace_bytes(int op, int64_t T, int64_t d_in, int64_t d_out, int64_t r, int dt, size_t* out_bytes) {
  if (!out_bytes || T < 0 || d_in < 0 || d_out < 0 || r < 0 || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  Arena ar{nullptr, 0, 0};
  switch (op) {
    case FLOP_OP_FWD:
    case FLOP_OP_COMPACT_FWD: plan_fwd_ws(ar, T, r, dt); break;
    case FLOP_OP_BWD: {   // large enough for the single call and for the grouped call (their split-K plans may differ)
      Arena g{nullptr, 0, 0};
      plan_bwd_ws(ar, T, d_in, d_out, r, dt, false);
      plan_bwd_ws(g, T, d_in, d_out, r, dt, true);
      ar.used = std::max(ar.used, g.used);
      break;
    }
    case FLOP_OP_L0: ar.used = l0_ws_bytes(T, r); break;
    case FLOP_OP_COMPACT: ar.used = 0; break;
    case FLOP_OP_EMBEDDING_BWD: ar.used = embedding_ws_bytes(T, r); break;
    default: return FLOP_ERR_INVALID_ARG;
  }
  *out_bytes = align_up(ar.used, 256);
  return FLOP_OK;
}

static int gate_sample_impl(const float* log_alpha, int64_t n, flop_hc_params_t hc, uint64_t seed, uint64_t offset,
                            const uint64_t* offset_dev, float* z, uint8_t* mask, float* dz_dla, void* stream) {
  if (n < 0 || !valid_hc(hc)) return FLOP_ERR_INVALID_ARG;
  if (n == 0) return FLOP_OK;
  if (!log_alpha || !z) return FLOP_ERR_INVALID_ARG;
  GateConsts g;
  g.beta_d = (double)hc.beta; g.gamma_d = (double)hc.gamma; g.zeta_d = (double)hc.zeta;
  g.inv_beta = (float)(1.0 / g.beta_d); g.neg_inv_beta_log2e = (float)(-1.4426950408889634 / g.beta_d); g.gamma = hc.gamma; g.zeta = hc.zeta;
  g.c0 = (float)(g.beta_d * log(-g.gamma_d / g.zeta_d));
  g.c1 = (float)(g.beta_d * log((1.0 - g.gamma_d) / (g.zeta_d - 1.0)));
  const int vec_ok = aligned16(log_alpha) && aligned16(z) && (!dz_dla || aligned16(dz_dla)) &&
                     (!mask || (reinterpret_cast<uintptr_t>(mask) & 3) == 0);
  const int64_t nblk = (n + 3) / 4;
  const int64_t want = (nblk + 255) / 256;
  const int grid = (int)std::min<int64_t>(want, (int64_t)num_sms() * 32);
  launch_k(gate_sample_kernel, dim3(grid), dim3(256), (size_t)(0), (cudaStream_t)stream, log_alpha, n, g, make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)),
                                                             offset, offset_dev, z, mask, dz_dla, vec_ok);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

int flop_gate_sample(const float* log_alpha, int64_t n, flop_hc_params_t hc, uint64_t seed, uint64_t offset, float* z,
                     uint8_t* mask, float* dz_dla, void* stream) {
  return gate_sample_impl(log_alpha, n, hc, seed, offset, nullptr, z, mask, dz_dla, stream);
}

int flop_gate_sample_devoff(const float* log_alpha, int64_t n, flop_hc_params_t hc, uint64_t seed, uint64_t offset,
                            const uint64_t* offset_dev, float* z, uint8_t* mask, float* dz_dla, void* stream) {
  if (!offset_dev) return FLOP_ERR_INVALID_ARG;
  return gate_sample_impl(log_alpha, n, hc, seed, offset, offset_dev, z, mask, dz_dla, stream);
}

static int fwd_impl(const void* X, int64_t ldx, const void* Q, int64_t ldq, const void* P, int64_t ldp, const float* z,
                    void* Y, int64_t ldy, void* H, int64_t ldh, int64_t T, int64_t d_in, int64_t d_out, int64_t r,
                    int dt, cudaStream_t st) {
  if (dt == FLOP_BF16) {
    if (r == 0 || d_in == 0) {
      FLOP_TRY(zero_2d<bf16>(Y, ldy, T, d_out, st));
      if (r > 0) FLOP_TRY(zero_2d<bf16>(H, ldh, T, r, st));
      return FLOP_OK;
    }
    if (T <= kSkinnyMaxT) {   // a few tokens: the weights are streamed once (CUDA cores up to 4 tokens, warp-level MMA up to 16)
      const int rc = launch_few_tokens(X, ldx, Q, ldq, H, ldh, z, T, r, d_in, st);
      if (rc == FLOP_OK) {
        const int rc2 = launch_few_tokens(H, ldh, P, ldp, Y, ldy, nullptr, T, d_out, r, st);
        if (rc2 != FLOP_ERR_UNSUPPORTED) return rc2;
      } else if (rc != FLOP_ERR_UNSUPPORTED) {
        return rc;
      }
    }
    // GEMM1: H' = (X Q^T) * z, gate applied to column k in the epilogue
    const TcPlan p1 = plan_tc(T, r, d_in, false, false);
    FLOP_TRY(launch_tc({X, ldx, false}, {Q, ldq, false}, T, r, d_in, p1, store_epilogue(H, ldh, z), st));
    // GEMM2: Y = H' P^T
    const TcPlan p2 = plan_tc(T, d_out, r, false, false);
    FLOP_TRY(launch_tc({H, ldh, false}, {P, ldp, false}, T, d_out, r, p2, store_epilogue(Y, ldy, nullptr), st));
  } else {
    FLOP_TRY(launch_simt((const float*)X, ldx, 1, (const float*)Q, ldq, 1, (float*)H, ldh, T, r, d_in, z, nullptr, 0, st));
    FLOP_TRY(launch_simt((const float*)H, ldh, 1, (const float*)P, ldp, 1, (float*)Y, ldy, T, d_out, r, nullptr, nullptr, 0, st));
  }
  return FLOP_OK;
}

int flop_gated_lowrank_fwd(const void* X, int64_t ldx, const void* Q, int64_t ldq, const void* P, int64_t ldp,
                           const float* z, void* Y, int64_t ldy, void* H_save, int64_t ldh, int64_t T, int64_t d_in,
                           int64_t d_out, int64_t r, int dt, void* ws, size_t ws_bytes, void* stream) {
  if (T < 0 || d_in < 0 || d_out < 0 || r < 0 || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  if (T == 0 || d_out == 0) return FLOP_OK;
  if (!check_mat(Y, ldy, d_out)) return FLOP_ERR_INVALID_ARG;
  if (r > 0 && (!z || !check_mat(P, ldp, r))) return FLOP_ERR_INVALID_ARG;
  if (r > 0 && d_in > 0 && (!check_mat(X, ldx, d_in) || !check_mat(Q, ldq, d_in))) return FLOP_ERR_INVALID_ARG;
  if (H_save && ldh < r) return FLOP_ERR_INVALID_ARG;
  void* H = H_save;
  if (!H && r > 0) {
    Arena ar{(unsigned char*)ws, ws_bytes, 0};
    Arena probe{nullptr, 0, 0};
    const size_t need = plan_fwd_ws(probe, T, r, dt).bytes;
    FLOP_TRY(check_ws(ws, ws_bytes, need));
    const FwdWs w = plan_fwd_ws(ar, T, r, dt);
    H = w.H; ldh = w.ldh;
  }
  if (dt == FLOP_BF16) {
    if (!bf16_ok(Y, ldy) || (r > 0 && (!bf16_ok(P, ldp) || !bf16_ok(H, ldh))) ||
        (r > 0 && d_in > 0 && (!bf16_ok(X, ldx) || !bf16_ok(Q, ldq))))
      return FLOP_ERR_UNSUPPORTED;
  }
  return fwd_impl(X, ldx, Q, ldq, P, ldp, z, Y, ldy, H, ldh, T, d_in, d_out, r, dt, (cudaStream_t)stream);
}

int flop_chain_fwd(const void* X, int64_t ldx, const void* Q, int64_t ldq, const void* P, int64_t ldp, const float* z, void* Y,
                   int64_t ldy, int64_t T, int64_t d_in, int64_t d_out, int64_t r, int dt, void* stream) {
  if (T < 0 || d_in < 0 || d_out < 0 || r < 0 || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  if (dt != FLOP_BF16) return FLOP_ERR_UNSUPPORTED;
  if (T == 0 || d_out == 0) return FLOP_OK;
  if (!check_mat(Y, ldy, d_out)) return FLOP_ERR_INVALID_ARG;
  if (!bf16_ok(Y, ldy)) return FLOP_ERR_UNSUPPORTED;
  if (r == 0 || d_in == 0) return zero_2d<bf16>(Y, ldy, T, d_out, (cudaStream_t)stream);
  if (!check_mat(X, ldx, d_in) || !check_mat(Q, ldq, d_in) || !check_mat(P, ldp, r)) return FLOP_ERR_INVALID_ARG;
  if (!bf16_ok(X, ldx) || !bf16_ok(Q, ldq) || !bf16_ok(P, ldp)) return FLOP_ERR_UNSUPPORTED;
  return launch_chain_fwd(X, ldx, Q, ldq, P, ldp, z, Y, ldy, T, d_in, d_out, r, (cudaStream_t)stream);
}

int flop_compact_fwd(const void* X, int64_t ldx, const void* Qc, int64_t ldqc, const void* Pc, int64_t ldpc, void* Y,
                     int64_t ldy, int64_t T, int64_t d_in, int64_t d_out, int64_t k, int dt, void* ws, size_t ws_bytes,
                     void* stream) {
  if (T < 0 || d_in < 0 || d_out < 0 || k < 0 || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  if (T == 0 || d_out == 0) return FLOP_OK;
  if (!check_mat(Y, ldy, d_out)) return FLOP_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (k == 0 || d_in == 0) {
    if (dt == FLOP_BF16) { if (!bf16_ok(Y, ldy)) return FLOP_ERR_UNSUPPORTED; return zero_2d<bf16>(Y, ldy, T, d_out, st); }
    return zero_2d<float>(Y, ldy, T, d_out, st);
  }
  if (!check_mat(X, ldx, d_in) || !check_mat(Qc, ldqc, d_in) || !check_mat(Pc, ldpc, k)) return FLOP_ERR_INVALID_ARG;
  Arena probe{nullptr, 0, 0};
  FLOP_TRY(check_ws(ws, ws_bytes, plan_fwd_ws(probe, T, k, dt).bytes));
  Arena ar{(unsigned char*)ws, ws_bytes, 0};
  const FwdWs w = plan_fwd_ws(ar, T, k, dt);
  if (dt == FLOP_BF16) {
    if (!bf16_ok(Y, ldy) || !bf16_ok(X, ldx) || !bf16_ok(Qc, ldqc) || !bf16_ok(Pc, ldpc)) return FLOP_ERR_UNSUPPORTED;
    if (T <= kSkinnyMaxT) {
      const int rc = launch_few_tokens(X, ldx, Qc, ldqc, w.H, w.ldh, nullptr, T, k, d_in, st);
      if (rc == FLOP_OK) {
        const int rc2 = launch_few_tokens(w.H, w.ldh, Pc, ldpc, Y, ldy, nullptr, T, d_out, k, st);
        if (rc2 != FLOP_ERR_UNSUPPORTED) return rc2;
      } else if (rc != FLOP_ERR_UNSUPPORTED) {
        return rc;
      }
    }
    const TcPlan p1 = plan_tc(T, k, d_in, false, false);
    FLOP_TRY(launch_tc({X, ldx, false}, {Qc, ldqc, false}, T, k, d_in, p1, store_epilogue(w.H, w.ldh, nullptr), st));
    const TcPlan p2 = plan_tc(T, d_out, k, false, false);
    FLOP_TRY(launch_tc({w.H, w.ldh, false}, {Pc, ldpc, false}, T, d_out, k, p2, store_epilogue(Y, ldy, nullptr), st));
  } else {
    FLOP_TRY(launch_simt((const float*)X, ldx, 1, (const float*)Qc, ldqc, 1, (float*)w.H, w.ldh, T, k, d_in, nullptr, nullptr, 0, st));
    FLOP_TRY(launch_simt((const float*)w.H, w.ldh, 1, (const float*)Pc, ldpc, 1, (float*)Y, ldy, T, d_out, k, nullptr, nullptr, 0, st));
  }
  return FLOP_OK;
}

int flop_gated_lowrank_bwd(const void* dY, int64_t lddy, const void* X, int64_t ldx, const void* Q, int64_t ldq,
                           const void* P, int64_t ldp, const float* z, const float* dz_dla, const void* H_save,
                           int64_t ldh, void* dX, int64_t lddx, void* dP, int64_t lddp, void* dQ, int64_t lddq,
                           float* dlog_alpha, int accumulate, int64_t T, int64_t d_in, int64_t d_out, int64_t r, int dt,
                           int wgrad_dt, void* ws, size_t ws_bytes, void* stream) {
  if (T < 0 || d_in < 0 || d_out < 0 || r < 0 || !valid_dt(dt) || !valid_dt(wgrad_dt)) return FLOP_ERR_INVALID_ARG;
  if (dt == FLOP_F32 && wgrad_dt != FLOP_F32) return FLOP_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  if (dX && lddx < d_in) return FLOP_ERR_INVALID_ARG;
  if (dP && lddp < r) return FLOP_ERR_INVALID_ARG;
  if (dQ && lddq < d_in) return FLOP_ERR_INVALID_ARG;
  if (dlog_alpha && r > 0 && !dz_dla) return FLOP_ERR_INVALID_ARG;
  const bool degenerate = T == 0 || r == 0 || d_in == 0 || d_out == 0;
  if (!degenerate) {
    if (!check_mat(dY, lddy, d_out) || !check_mat(X, ldx, d_in) || !check_mat(Q, ldq, d_in) || !check_mat(P, ldp, r) ||
        !z || !check_mat(H_save, ldh, r))
      return FLOP_ERR_INVALID_ARG;
  }
  if (dt == FLOP_BF16) {
    if ((dX && !bf16_ok(dX, lddx)) || (!degenerate && (!bf16_ok(dY, lddy) || !bf16_ok(X, ldx) || !bf16_ok(Q, ldq) ||
                                                       !bf16_ok(P, ldp) || !bf16_ok(H_save, ldh))))
      return FLOP_ERR_UNSUPPORTED;
  }
  if (degenerate) {
    // every product is empty: gradients are zero (or unchanged when accumulating)
    if (dX && T > 0 && d_in > 0) FLOP_TRY(dt == FLOP_BF16 ? zero_2d<bf16>(dX, lddx, T, d_in, st) : zero_2d<float>(dX, lddx, T, d_in, st));
    if (!accumulate) {
      if (dP) FLOP_TRY(wgrad_dt == FLOP_BF16 ? zero_2d<bf16>(dP, lddp, d_out, r, st) : zero_2d<float>(dP, lddp, d_out, r, st));
      if (dQ) FLOP_TRY(wgrad_dt == FLOP_BF16 ? zero_2d<bf16>(dQ, lddq, r, d_in, st) : zero_2d<float>(dQ, lddq, r, d_in, st));
      if (dlog_alpha) FLOP_TRY(zero_2d<float>(dlog_alpha, r, 1, r, st));
    }
    return FLOP_OK;
  }
  Arena probe{nullptr, 0, 0};
  FLOP_TRY(check_ws(ws, ws_bytes, plan_bwd_ws(probe, T, d_in, d_out, r, dt).bytes));
  Arena ar{(unsigned char*)ws, ws_bytes, 0};
  const BwdWs w = plan_bwd_ws(ar, T, d_in, d_out, r, dt);
  const bool need_m = dQ || dlog_alpha;   // M = dH'^T X feeds both dQ and dz

  if (dt == FLOP_BF16) {
    // dH' = dY P            (A = dY K-major over d_out; B(n=k_rank, k=i) = P[i, k_rank]: MN-major)
    const TcPlan ph = plan_tc(T, r, d_out, false, true);
    FLOP_TRY(launch_tc({dY, lddy, false}, {P, ldp, true}, T, r, d_out, ph, store_epilogue(w.dH, w.lddh, nullptr), st));
    // A weight-gradient GEMM that needs no split-K writes its result straight from the epilogue;
    // otherwise it writes fp32 slices that the finishing kernel adds up in order.
    const bool direct_p = dP && w.plan_p.splits == 1 && wgrad_direct_ok(dP, lddp, wgrad_dt);
    const bool direct_q = need_m && w.plan_q.splits == 1 && (!dQ || wgrad_direct_ok(dQ, lddq, wgrad_dt));
    if (dP) {
      // dP = dY^T H'        (contract over tokens: both operands MN-major)
      TcEpilogue e{};
      if (direct_p) e = wgrad_epilogue(dP, lddp, wgrad_dt, nullptr, accumulate);
      else { e.kind = tc::EPI_SLICE; e.slices = w.slices_p; e.slice_elems = w.slice_elems_p; e.ld_slice = w.ld_slice_p; }
      FLOP_TRY(launch_tc({dY, lddy, true}, {H_save, ldh, true}, d_out, r, T, w.plan_p, e, st));
    }
    if (need_m) {
      // M = dH'^T X; dQ = diag(z) M; dz_k = <Q[k,:], M[k,:]> fused into the GEMM epilogue per tile
      TcEpilogue e{};
      if (direct_q) e = dQ ? wgrad_epilogue(dQ, lddq, wgrad_dt, z, accumulate) : wgrad_epilogue(w.slices_q, w.ld_slice_q, FLOP_F32, nullptr, 0);
      else { e.kind = tc::EPI_SLICE; e.slices = w.slices_q; e.slice_elems = w.slice_elems_q; e.ld_slice = w.ld_slice_q; }
      if (dlog_alpha) { e.qdot = (const bf16*)Q; e.ldq = ldq; e.dz_part = w.dz_part; e.dz_stride = r; }
      FLOP_TRY(launch_tc({w.dH, w.lddh, true}, {X, ldx, true}, r, d_in, T, w.plan_q, e, st));
    }
    {
      // one launch: ordered split-K sums -> dP, diag(z)-scaled dQ; diag(z) Q for the dX GEMM; dlog_alpha
      BwdFinishArgs a{};
      a.slices_p = w.slices_p; a.n_slices_p = w.plan_p.splits; a.slice_elems_p = w.slice_elems_p; a.ld_slice_p = w.ld_slice_p;
      a.d_out = (int)d_out; a.r = (int)r; a.dP = direct_p ? nullptr : dP; a.lddp = lddp;
      a.slices_q = w.slices_q; a.n_slices_q = w.plan_q.splits; a.slice_elems_q = w.slice_elems_q; a.ld_slice_q = w.ld_slice_q;
      a.d_in = (int)d_in; a.dQ = direct_q ? nullptr : dQ; a.lddq = lddq; a.z = z;
      a.Q = (const bf16*)Q; a.ldq = ldq; a.Qz = dX ? (bf16*)w.Qz : nullptr; a.ldqz = w.ldqz;
      a.dz_part = w.dz_part; a.n_part = w.n_part; a.dz_dla = dz_dla; a.dlog_alpha = dlog_alpha; a.accumulate = accumulate;
      const int64_t units = bwd_finish_units(a);
      if (units > 0) {
        const int grid = (int)std::min<int64_t>((units + 255) / 256, (int64_t)num_sms() * 8);
        if (wgrad_dt == FLOP_BF16) launch_k(bwd_finish_kernel<bf16>, dim3(grid), dim3(256), (size_t)(0), st, a);
        else                       launch_k(bwd_finish_kernel<float>, dim3(grid), dim3(256), (size_t)(0), st, a);
        count_launch();
        FLOP_CUDA(cudaGetLastError());
      }
    }
    if (dX) {
      // dX = dH' (diag(z) Q)   (B(n=j, k=k_rank) = Qz[k_rank, j]: MN-major)
      const TcPlan px = plan_tc(T, d_in, r, false, true);
      FLOP_TRY(launch_tc({w.dH, w.lddh, false}, {w.Qz, w.ldqz, true}, T, d_in, r, px, store_epilogue(dX, lddx, nullptr), st));
    }
  } else {
    const float* dYf = (const float*)dY; const float* Xf = (const float*)X; const float* Qf = (const float*)Q;
    const float* Pf = (const float*)P; const float* Hf = (const float*)H_save;
    float* dHf = (float*)w.dH;
    // dH'[t,k] = sum_i dY[t,i] P[i,k]
    FLOP_TRY(launch_simt(dYf, lddy, 1, Pf, 1, ldp, dHf, w.lddh, T, r, d_out, nullptr, nullptr, 0, st));
    // dP[i,k] = sum_t dY[t,i] H'[t,k]
    if (dP) FLOP_TRY(launch_simt(dYf, 1, lddy, Hf, 1, ldh, (float*)dP, lddp, d_out, r, T, nullptr, nullptr, accumulate, st));
    if (need_m) {
      // M[k,j] = sum_t dH'[t,k] X[t,j] into the slice buffer, then the same finalisation as the tensor-core path
      FLOP_TRY(launch_simt(dHf, 1, w.lddh, Xf, 1, ldx, w.slices_q, w.ld_slice_q, r, d_in, T, nullptr, nullptr, 0, st));
      FLOP_TRY((finalize_wgrad<float, float>(w.slices_q, 1, w.slice_elems_q, w.ld_slice_q, r, d_in, z, dQ, lddq, accumulate,
                                             dlog_alpha ? Q : nullptr, ldq, w.dz_part, st)));
      if (dlog_alpha) {
        launch_k(dalpha_kernel, dim3((unsigned)((r + 255) / 256)), dim3(256), (size_t)(0), st, w.dz_part, 1, r, dz_dla, (int)r, dlog_alpha, accumulate);
        count_launch();
        FLOP_CUDA(cudaGetLastError());
      }
    }
    if (dX) {
      launch_k(scale_rows_kernel<float>, dim3((unsigned)r), dim3(256), (size_t)(0), st, Qf, ldq, z, (int)r, (int)d_in, (float*)w.Qz, w.ldqz);
      count_launch();
      FLOP_CUDA(cudaGetLastError());
      // dX[t,j] = sum_k dH'[t,k] Qz[k,j]
      FLOP_TRY(launch_simt(dHf, w.lddh, 1, (const float*)w.Qz, 1, w.ldqz, (float*)dX, lddx, T, d_in, r, nullptr, nullptr, 0, st));
    }
  }
  return FLOP_OK;
}

static int check_sync(const void* sync, size_t sync_bytes) {
  if (!sync) return FLOP_OK;
  if ((reinterpret_cast<uintptr_t>(sync) & 15) != 0 || sync_bytes < kSyncBytes) return FLOP_ERR_WORKSPACE;
  return FLOP_OK;
}

static int fwd_grouped_impl(const flop_fwd_problem_t* pr, int n, int dt, void* sync, size_t sync_bytes, void* stream) {
  if (n < 0 || (n > 0 && !pr) || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  FLOP_TRY(check_sync(sync, sync_bytes));
  bool grouped = dt == FLOP_BF16;
  for (int i = 0; i < n; ++i) {
    const flop_fwd_problem_t& a = pr[i];
    if (a.T < 0 || a.d_in < 0 || a.d_out < 0 || a.r < 0) return FLOP_ERR_INVALID_ARG;
    if (a.T > 0 && a.r > 0 && !a.H_save) return FLOP_ERR_INVALID_ARG;   // the grouped call has no scratch: H' goes to H_save
    if (a.T == 0 || a.d_in == 0 || a.d_out == 0 || a.r == 0) grouped = false;
  }
  if (!grouped) {   // fp32 storage or an empty problem: one call per problem
    for (int i = 0; i < n; ++i) {
      const flop_fwd_problem_t& a = pr[i];
      if (a.r_dev) return FLOP_ERR_UNSUPPORTED;   // a device-side rank needs the grouped bf16 kernels
      FLOP_TRY(flop_gated_lowrank_fwd(a.X, a.ldx, a.Q, a.ldq, a.P, a.ldp, a.z, a.Y, a.ldy, a.H_save, a.ldh, a.T, a.d_in, a.d_out,
                                      a.r, dt, nullptr, 0, stream));
    }
    return FLOP_OK;
  }
  std::vector<TcJob> g1, g2;
  std::vector<Mnk> m1, m2;
  for (int i = 0; i < n; ++i) {
    m1.push_back({pr[i].T, pr[i].r, pr[i].d_in});
    m2.push_back({pr[i].T, pr[i].d_out, pr[i].r});
  }
  const GroupShape s1 = plan_group(m1, false), s2 = plan_group(m2, false);
  for (int i = 0; i < n; ++i) {
    const flop_fwd_problem_t& a = pr[i];
    if (!check_mat(a.Y, a.ldy, a.d_out) || !a.z || !check_mat(a.P, a.ldp, a.r) || !check_mat(a.X, a.ldx, a.d_in) ||
        !check_mat(a.Q, a.ldq, a.d_in) || a.ldh < a.r)
      return FLOP_ERR_INVALID_ARG;
    if (!bf16_ok(a.Y, a.ldy) || !bf16_ok(a.P, a.ldp) || !bf16_ok(a.H_save, a.ldh) || !bf16_ok(a.X, a.ldx) || !bf16_ok(a.Q, a.ldq))
      return FLOP_ERR_UNSUPPORTED;
    TcJob j1{{a.X, a.ldx, false}, {a.Q, a.ldq, false}, a.T, a.r, a.d_in, fixed_plan(a.T, a.r, a.d_in, s1.bn, s1.cta2),
             store_epilogue(a.H_save, a.ldh, a.z)};
    TcJob j2{{a.H_save, a.ldh, false}, {a.P, a.ldp, false}, a.T, a.d_out, a.r, fixed_plan(a.T, a.d_out, a.r, s2.bn, s2.cta2),
             store_epilogue(a.Y, a.ldy, nullptr)};
    j1.dyn_n = a.r_dev;   // only the first *r_dev rank components exist this step
    j2.dyn_k = a.r_dev;
    g1.push_back(j1);
    g2.push_back(j2);
  }
  cudaStream_t st = (cudaStream_t)stream;
  // One launch for both products when the caller brought a sync area: every problem's first product publishes
  // its 256-row blocks of H', the tiles of the second wait for the block they read.
  {
    size_t words = tc::kSyncFixed;
    std::vector<TcJob> all;
    std::vector<int> dep_job;
    for (int i = 0; i < n; ++i) {
      TcJob j = g1[(size_t)i];
      j.stage = 0; j.order_class = 0;
      j.link.sig = (unsigned*)sync + words;
      words += (size_t)j.pl.tiles_m;
      all.push_back(j);
      dep_job.push_back(-1);
    }
    for (int i = 0; i < n; ++i) {
      TcJob j = g2[(size_t)i];
      const TcJob& src = all[(size_t)i];
      j.stage = 1; j.order_class = 0;
      j.link.dep = src.link.sig; j.link.dep_mode = 1;
      j.link.dep_n_cap = (int)src.N; j.link.dep_bn = src.pl.bn; j.link.dep_dyn_n = src.dyn_n;
      all.push_back(j);
      dep_job.push_back(i);
    }
    if (chain_ok(all, sync, sync_bytes, words)) {
      if (tuning().chain_stages >= 2) return launch_tc_chain(all, dep_job, (unsigned*)sync, (int)words, false, st);
      // a launch per product, each drawing its tiles from a queue (nothing waits inside a launch)
      const std::vector<int> none((size_t)n, -1);
      FLOP_TRY(launch_tc_chain(g1, none, (unsigned*)sync, tc::kSyncFixed, false, st));
      return launch_tc_chain(g2, none, (unsigned*)sync, tc::kSyncFixed, false, st);
    }
  }
  FLOP_TRY(launch_tc_group(g1, st));   // H' = (X Q^T) * z for every problem
  FLOP_TRY(launch_tc_group(g2, st));   // Y = H' P^T
  return FLOP_OK;
}

int flop_gated_lowrank_fwd_grouped(const flop_fwd_problem_t* pr, int n, int dt, void* stream) {
  return fwd_grouped_impl(pr, n, dt, nullptr, 0, stream);
}

int flop_gated_lowrank_fwd_chained(const flop_fwd_problem_t* pr, int n, int dt, void* sync, size_t sync_bytes, void* stream) {
  if (!sync) return FLOP_ERR_WORKSPACE;
  return fwd_grouped_impl(pr, n, dt, sync, sync_bytes, stream);
}

int flop_sync_bytes(size_t* out_bytes) {
  if (!out_bytes) return FLOP_ERR_INVALID_ARG;
  *out_bytes = kSyncBytes;
  return FLOP_OK;
}

static int bwd_grouped_impl(const flop_bwd_problem_t* pr, int n, int accumulate, int dt, int wgrad_dt, void* sync,
                            size_t sync_bytes, void* stream) {
  if (n < 0 || (n > 0 && !pr) || !valid_dt(dt) || !valid_dt(wgrad_dt)) return FLOP_ERR_INVALID_ARG;
  FLOP_TRY(check_sync(sync, sync_bytes));
  if (dt == FLOP_F32 && wgrad_dt != FLOP_F32) return FLOP_ERR_UNSUPPORTED;
  bool grouped = dt == FLOP_BF16;
  for (int i = 0; i < n; ++i) {
    const flop_bwd_problem_t& a = pr[i];
    if (a.T < 0 || a.d_in < 0 || a.d_out < 0 || a.r < 0) return FLOP_ERR_INVALID_ARG;
    if (a.T == 0 || a.d_in == 0 || a.d_out == 0 || a.r == 0) grouped = false;
  }
  if (!grouped) {
    for (int i = 0; i < n; ++i) {
      const flop_bwd_problem_t& a = pr[i];
      if (a.r_dev || a.defer_dlog_alpha) return FLOP_ERR_UNSUPPORTED;
      FLOP_TRY(flop_gated_lowrank_bwd(a.dY, a.lddy, a.X, a.ldx, a.Q, a.ldq, a.P, a.ldp, a.z, a.dz_dla, a.H_save, a.ldh, a.dX,
                                      a.lddx, a.dP, a.lddp, a.dQ, a.lddq, a.dlog_alpha, accumulate, a.T, a.d_in, a.d_out, a.r, dt,
                                      wgrad_dt, a.ws, a.ws_bytes, stream));
    }
    return FLOP_OK;
  }
  cudaStream_t st = (cudaStream_t)stream;
  std::vector<TcJob> g3, g4, g5, g6;
  std::vector<BwdFinishArgs> fin;
  std::vector<BwdWs> wss;
  bool direct = true;   // weight gradients straight from the GEMM epilogue (no split-K, no fp32 slices)
  for (int i = 0; i < n; ++i) {
    const flop_bwd_problem_t& a = pr[i];
    if ((a.dX && a.lddx < a.d_in) || (a.dP && a.lddp < a.r) || (a.dQ && a.lddq < a.d_in) || (a.dlog_alpha && !a.dz_dla))
      return FLOP_ERR_INVALID_ARG;
    if (!check_mat(a.dY, a.lddy, a.d_out) || !check_mat(a.X, a.ldx, a.d_in) || !check_mat(a.Q, a.ldq, a.d_in) ||
        !check_mat(a.P, a.ldp, a.r) || !a.z || !check_mat(a.H_save, a.ldh, a.r))
      return FLOP_ERR_INVALID_ARG;
    if (a.Qz && a.ldqz < a.d_in) return FLOP_ERR_INVALID_ARG;
    if ((a.dX && !bf16_ok(a.dX, a.lddx)) || !bf16_ok(a.dY, a.lddy) || !bf16_ok(a.X, a.ldx) || !bf16_ok(a.Q, a.ldq) ||
        !bf16_ok(a.P, a.ldp) || !bf16_ok(a.H_save, a.ldh) || (a.Qz && !bf16_ok(a.Qz, a.ldqz)))
      return FLOP_ERR_UNSUPPORTED;
    Arena probe{nullptr, 0, 0};
    FLOP_TRY(check_ws(a.ws, a.ws_bytes, plan_bwd_ws(probe, a.T, a.d_in, a.d_out, a.r, dt, true).bytes));
    Arena ar{(unsigned char*)a.ws, a.ws_bytes, 0};
    wss.push_back(plan_bwd_ws(ar, a.T, a.d_in, a.d_out, a.r, dt, true));
    if ((a.dP && !wgrad_direct_ok(a.dP, a.lddp, wgrad_dt)) || (a.dQ && !wgrad_direct_ok(a.dQ, a.lddq, wgrad_dt))) direct = false;
  }
  // One tile shape per stage for all problems of the call.  The weight gradients go direct when
  // the un-split work items fill the machine at least once.
  std::vector<Mnk> m3, mw, m6;
  for (int i = 0; i < n; ++i) {
    const flop_bwd_problem_t& a = pr[i];
    m3.push_back({a.T, a.r, a.d_out});
    if (a.dP) mw.push_back({a.d_out, a.r, a.T});
    if (a.dQ || a.dlog_alpha) mw.push_back({a.r, a.d_in, a.T});
    if (a.dX) m6.push_back({a.T, a.d_in, a.r});
  }
  const GroupShape s3 = plan_group(m3, true), s6 = plan_group(m6, true);
  // When the activation-gradient products run on CTA pairs, the weight gradients take pair tiles too if those
  // fill the machine, so that each can share a launch with them (see below): at Transformer-XL sizes the cost
  // model alone prefers one-CTA 128 x 128 tiles by half a per cent, and the shared launches are 16 % faster.
  GroupShape sw = plan_group(mw, true, true);
  if (!sw.cta2 && s3.cta2 && (m6.empty() || s6.cta2)) {
    const GroupShape swp = plan_group(mw, true, true, true);
    if (swp.bn != 0 && swp.items >= num_sms() / 2) sw = swp;
  }
  if (sw.bn == 0 || sw.items < (sw.cta2 ? num_sms() / 2 : num_sms())) direct = false;
  auto direct_plan = [&](int64_t M, int64_t N, int64_t K) { return fixed_plan(M, N, K, sw.bn, sw.cta2); };
  for (int i = 0; i < n; ++i) {
    const flop_bwd_problem_t& a = pr[i];
    const BwdWs& w = wss[i];
    const bool need_m = a.dQ || a.dlog_alpha;
    TcJob j3{{a.dY, a.lddy, false}, {a.P, a.ldp, true}, a.T, a.r, a.d_out, fixed_plan(a.T, a.r, a.d_out, s3.bn, s3.cta2),
             store_epilogue(w.dH, w.lddh, nullptr)};
    j3.dyn_n = a.r_dev;
    g3.push_back(j3);
    int n_part = w.n_part;
    if (a.dP) {
      if (direct) {
        TcJob j{{a.dY, a.lddy, true}, {a.H_save, a.ldh, true}, a.d_out, a.r, a.T, direct_plan(a.d_out, a.r, a.T),
                wgrad_epilogue(a.dP, a.lddp, wgrad_dt, nullptr, accumulate)};
        j.dyn_n = a.r_dev;
        g4.push_back(j);
      } else {
        TcEpilogue e{};
        e.kind = tc::EPI_SLICE; e.slices = w.slices_p; e.slice_elems = w.slice_elems_p; e.ld_slice = w.ld_slice_p;
        TcJob j{{a.dY, a.lddy, true}, {a.H_save, a.ldh, true}, a.d_out, a.r, a.T, w.plan_p, e};
        j.dyn_n = a.r_dev;
        g4.push_back(j);
      }
    }
    if (need_m) {
      TcEpilogue e{};
      TcPlan pl = w.plan_q;
      if (direct) {
        // dQ = diag(z) (dH'^T X) stored in place (dQ may be absent when only dlog_alpha is wanted: then
        // the product still runs for the fused row dots and its values go to the slice buffer)
        pl = direct_plan(a.r, a.d_in, a.T);
        if (a.dQ) e = wgrad_epilogue(a.dQ, a.lddq, wgrad_dt, a.z, accumulate);
        else      e = wgrad_epilogue(w.slices_q, w.ld_slice_q, FLOP_F32, nullptr, 0);
        n_part = 2 * pl.tiles_n;
      } else {
        e.kind = tc::EPI_SLICE; e.slices = w.slices_q; e.slice_elems = w.slice_elems_q; e.ld_slice = w.ld_slice_q;
      }
      if (a.dlog_alpha) { e.qdot = (const bf16*)a.Q; e.ldq = a.ldq; e.dz_part = w.dz_part; e.dz_stride = a.r; e.dz_meta = a.defer_dlog_alpha ? w.dz_meta : nullptr; }
      TcJob j5{{w.dH, w.lddh, true}, {a.X, a.ldx, true}, a.r, a.d_in, a.T, pl, e};
      j5.dyn_m = a.r_dev;
      g5.push_back(j5);
    }
    BwdFinishArgs f{};
    f.slices_p = w.slices_p; f.n_slices_p = w.plan_p.splits; f.slice_elems_p = w.slice_elems_p; f.ld_slice_p = w.ld_slice_p;
    f.d_out = (int)a.d_out; f.r = (int)a.r; f.dP = direct ? nullptr : a.dP; f.lddp = a.lddp;
    f.slices_q = w.slices_q; f.n_slices_q = w.plan_q.splits; f.slice_elems_q = w.slice_elems_q; f.ld_slice_q = w.ld_slice_q;
    f.d_in = (int)a.d_in; f.dQ = direct ? nullptr : a.dQ; f.lddq = a.lddq; f.z = a.z;
    // diag(z) Q: the caller's (formed once per step by flop_scale_rows_grouped), else formed here in the workspace
    f.Q = (const bf16*)a.Q; f.ldq = a.ldq; f.Qz = (a.dX && !a.Qz) ? (bf16*)w.Qz : nullptr; f.ldqz = w.ldqz;
    f.dz_part = w.dz_part; f.n_part = n_part; f.dz_dla = a.dz_dla; f.dlog_alpha = a.defer_dlog_alpha ? nullptr : a.dlog_alpha; f.accumulate = accumulate;
    fin.push_back(f);
    if (a.dX) {
      TcJob j6{{w.dH, w.lddh, false}, {a.Qz ? a.Qz : w.Qz, a.Qz ? a.ldqz : w.ldqz, true}, a.T, a.d_in, a.r, fixed_plan(a.T, a.d_in, a.r, s6.bn, s6.cta2),
               store_epilogue(a.dX, a.lddx, nullptr)};
      j6.dyn_k = a.r_dev;
      g6.push_back(j6);
    }
  }
  auto run_finish = [&](const std::vector<BwdFinishArgs>& list) -> int {
    for (size_t i = 0; i < list.size(); i += kFinishGroup) {
      BwdFinishGroup g;
      memset(&g, 0, sizeof(g));
      for (; g.n < kFinishGroup && i + g.n < list.size(); ++g.n) {
        g.a[g.n] = list[i + g.n];
        g.unit_begin[g.n + 1] = g.unit_begin[g.n] + bwd_finish_units(g.a[g.n]);
      }
      const int64_t units = g.unit_begin[g.n];
      if (units > 0) {
        const int grid = (int)std::min<int64_t>((units + 255) / 256, (int64_t)num_sms() * 8);
        if (wgrad_dt == FLOP_BF16) launch_k(bwd_finish_group_kernel<bf16>, dim3(grid), dim3(256), (size_t)0, st, g);
        else                       launch_k(bwd_finish_group_kernel<float>, dim3(grid), dim3(256), (size_t)0, st, g);
        count_launch();
        FLOP_CUDA(cudaGetLastError());
      }
    }
    return FLOP_OK;
  };
  // Two balanced launches instead of three uneven ones (gemm_tc2_dual.cuh): the products that need only saved
  // tensors (dH' = dY P and dP = dY^T H') share the first work list, those that need dH' (dQ with the fused
  // <Q, .> row dots, and dX) the second.  diag(z) Q depends on nothing computed here and is formed first; the
  // ordered second stage of dlog_alpha comes last.
  const int merge_on = tuning().stage_merge;
  const bool pairs_everywhere = !g3.empty() && g3[0].pl.cta2 && (g4.empty() || g4[0].pl.cta2) && (g5.empty() || g5[0].pl.cta2) &&
                                (g6.empty() || g6[0].pl.cta2);
  // With a sync area: the whole backward pass of the call in ONE launch.  dH' tiles publish their row blocks;
  // dX tiles wait for the block they read and for diag(z) Q, which the launch forms as side work; dQ tiles wait
  // block by block as their contraction over the tokens advances, and the last tile of every 32-row slab of dQ
  // adds up the slab's dlog_alpha partials.  No small kernel before or after.
  if (direct && pairs_everywhere && sync) {
    size_t words = tc::kSyncFixed;
    std::vector<TcJob> all;
    std::vector<int> dep_job;
    // queue order: dH' tiles (everything else waits for them), the long dP tiles, the long dQ tiles (by then all of
    // dH' is written), and the short dX tiles last, so that the launch ends on short tiles
    for (size_t i = 0; i < g3.size(); ++i) {     // one dH' job per problem, in problem order
      TcJob j = g3[i];
      j.stage = 0; j.order_class = 0;
      j.link.sig = (unsigned*)sync + words;
      words += (size_t)j.pl.tiles_m;
      all.push_back(j);
      dep_job.push_back(-1);
    }
    for (TcJob j : g4) { j.stage = 0; j.order_class = 1; all.push_back(j); dep_job.push_back(-1); }
    // g5 / g6 hold one job per problem that asked for dQ or dlog_alpha / for dX, in problem order
    size_t i6 = 0, i5 = 0;
    for (int i = 0; i < n; ++i) {
      const flop_bwd_problem_t& a = pr[i];
      const TcJob& src = all[(size_t)i];
      if (a.dQ || a.dlog_alpha) {
        TcJob j = g5[i5++];
        j.stage = 1; j.order_class = 0;
        j.link.dep = src.link.sig; j.link.dep_mode = 2;
        j.link.dep_n_cap = (int)src.N; j.link.dep_bn = src.pl.bn; j.link.dep_dyn_n = src.dyn_n;
        if (a.dlog_alpha && !a.defer_dlog_alpha) {
          j.link.fin = (unsigned*)sync + words;
          words += (size_t)j.pl.tiles_m * 8;
          j.link.dz_dla = a.dz_dla; j.link.dla = a.dlog_alpha; j.link.dla_accumulate = accumulate;
        }
        all.push_back(j);
        dep_job.push_back(i);
      }
    }
    for (int i = 0; i < n; ++i) {
      const flop_bwd_problem_t& a = pr[i];
      const TcJob& src = all[(size_t)i];
      if (a.dX) {
        TcJob j = g6[i6++];
        j.stage = 1; j.order_class = 1;
        j.link.dep = src.link.sig; j.link.dep_mode = 1;
        j.link.dep_n_cap = (int)src.N; j.link.dep_bn = src.pl.bn; j.link.dep_dyn_n = src.dyn_n;
        if (!a.Qz) {     // no diag(z) Q from the caller: the launch's helper warps form it in the workspace
          j.link.side_dep = 1;
          j.link.sw_q = (const bf16*)a.Q; j.link.sw_ldq = a.ldq; j.link.sw_qz = (bf16*)wss[(size_t)i].Qz; j.link.sw_ldqz = wss[(size_t)i].ldqz;
          j.link.sw_z = a.z; j.link.sw_rows = (int)a.r; j.link.sw_cols = (int)a.d_in;
        }
        all.push_back(j);
        dep_job.push_back(i);
      }
    }
    if (chain_ok(all, sync, sync_bytes, words)) {
      if (tuning().chain_stages >= 2) return launch_tc_chain(all, dep_job, (unsigned*)sync, (int)words, true, st);
      // Two launches (dH' with dP, then dQ with dX), each drawing its tiles from a queue; nothing waits inside a
      // launch.  The second still finishes dlog_alpha by itself; diag(z) Q comes from the caller, else from the
      // small kernel before the first launch.
      std::vector<TcJob> one, two;
      for (TcJob j : all) {
        const bool second = j.stage != 0;
        j.stage = 0; j.order_class = 0;      // no waits inside a launch: long tiles first
        j.link.sig = nullptr; j.link.dep = nullptr; j.link.dep_mode = 0; j.link.side_dep = 0; j.link.sw_qz = nullptr;
        (second ? two : one).push_back(j);
      }
      bool need_pre = false;
      std::vector<BwdFinishArgs> pre = fin;
      for (size_t i = 0; i < pre.size(); ++i) {
        pre[i].dlog_alpha = nullptr;
        if (pre[i].Qz) need_pre = true;
      }
      if (need_pre) FLOP_TRY(run_finish(pre));
      FLOP_TRY(launch_tc_chain(one, std::vector<int>(one.size(), -1), (unsigned*)sync, tc::kSyncFixed, true, st));
      if (!two.empty()) FLOP_TRY(launch_tc_chain(two, std::vector<int>(two.size(), -1), (unsigned*)sync, (int)words, true, st));
      return FLOP_OK;
    }
  }
  if (direct && merge_on && pairs_everywhere && g3.size() + g4.size() <= (size_t)tc::kMaxGroup &&
      g5.size() + g6.size() <= (size_t)tc::kMaxGroup) {
    std::vector<BwdFinishArgs> pre = fin, post = fin;
    for (auto& f : pre) f.dlog_alpha = nullptr;
    for (auto& f : post) f.Qz = nullptr;
    FLOP_TRY(run_finish(pre));
    g3.insert(g3.end(), g4.begin(), g4.end());
    FLOP_TRY(launch_tc_group(g3, st));
    g5.insert(g5.end(), g6.begin(), g6.end());
    FLOP_TRY(launch_tc_group(g5, st));
    FLOP_TRY(run_finish(post));
    return FLOP_OK;
  }
  if (direct) {   // both weight-gradient products of every matrix in one work list
    g4.insert(g4.end(), g5.begin(), g5.end());
    g5.clear();
  }
  FLOP_TRY(launch_tc_group(g3, st));   // dH' = dY P
  FLOP_TRY(launch_tc_group(g4, st));   // dY^T H' slices
  FLOP_TRY(launch_tc_group(g5, st));   // dH'^T X slices + fused <Q, .> row dots
  FLOP_TRY(run_finish(fin));
  FLOP_TRY(launch_tc_group(g6, st));   // dX = dH' (diag(z) Q)
  return FLOP_OK;
}

int flop_gated_lowrank_bwd_grouped(const flop_bwd_problem_t* pr, int n, int accumulate, int dt, int wgrad_dt, void* stream) {
  return bwd_grouped_impl(pr, n, accumulate, dt, wgrad_dt, nullptr, 0, stream);
}

int flop_gated_lowrank_bwd_chained(const flop_bwd_problem_t* pr, int n, int accumulate, int dt, int wgrad_dt, void* sync,
                                   size_t sync_bytes, void* stream) {
  if (!sync) return FLOP_ERR_WORKSPACE;
  return bwd_grouped_impl(pr, n, accumulate, dt, wgrad_dt, sync, sync_bytes, stream);
}

int flop_dlog_alpha_finish_grouped(const flop_bwd_problem_t* pr, int n, int accumulate, int dt, void* stream) {
  if (n < 0 || (n > 0 && !pr) || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  if (dt != FLOP_BF16) return FLOP_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  for (int i0 = 0; i0 < n; i0 += kDlaGroup) {
    DlaFinishGroup g;
    memset(&g, 0, sizeof(g));
    int max_r = 0;
    for (; g.n < kDlaGroup && i0 + g.n < n; ++g.n) {
      const flop_bwd_problem_t& a = pr[i0 + g.n];
      if (a.T < 0 || a.d_in < 0 || a.d_out < 0 || a.r < 0 || a.r > INT32_MAX) return FLOP_ERR_INVALID_ARG;
      DlaFinish& o = g.a[g.n];
      if (!a.dlog_alpha || a.T == 0 || a.r == 0 || a.d_in == 0 || a.d_out == 0) { o.r = 0; continue; }
      if (!a.dz_dla) return FLOP_ERR_INVALID_ARG;
      Arena probe{nullptr, 0, 0};
      FLOP_TRY(check_ws(a.ws, a.ws_bytes, plan_bwd_ws(probe, a.T, a.d_in, a.d_out, a.r, dt, true).bytes));
      Arena ar{(unsigned char*)a.ws, a.ws_bytes, 0};
      const BwdWs w = plan_bwd_ws(ar, a.T, a.d_in, a.d_out, a.r, dt, true);
      o.dz_part = w.dz_part; o.n_part = w.dz_meta; o.cap = (int)std::max<int64_t>(w.n_part, 2 * ((a.d_in + 63) / 64));
      o.dz_dla = a.dz_dla; o.dla = a.dlog_alpha; o.r = (int)a.r;
      max_r = std::max(max_r, o.r);
    }
    if (max_r == 0) continue;
    launch_k(dalpha_group_kernel, dim3((unsigned)((max_r + 255) / 256), (unsigned)g.n), dim3(256), (size_t)0, st, g, accumulate);
    count_launch();
    FLOP_CUDA(cudaGetLastError());
  }
  return FLOP_OK;
}

int flop_scale_rows_grouped(const flop_scale_rows_t* pr, int n, int dt, void* stream) {
  if (n < 0 || (n > 0 && !pr) || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  if (dt != FLOP_BF16) return FLOP_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  for (int i0 = 0; i0 < n; i0 += kScaleGroup) {
    ScaleRowsGroup g;
    memset(&g, 0, sizeof(g));
    int64_t max_units = 0;
    for (; g.n < kScaleGroup && i0 + g.n < n; ++g.n) {
      const flop_scale_rows_t& a = pr[i0 + g.n];
      if (a.r < 0 || a.d_in < 0 || a.r > INT32_MAX || a.d_in > INT32_MAX) return FLOP_ERR_INVALID_ARG;
      if (a.r > 0 && a.d_in > 0 && (!a.Q || !a.z || !a.Qz || a.ldq < a.d_in || a.ldqz < a.d_in)) return FLOP_ERR_INVALID_ARG;
      if (a.r > 0 && a.d_in > 0 && (!bf16_ok(a.Q, a.ldq) || !bf16_ok(a.Qz, a.ldqz))) return FLOP_ERR_UNSUPPORTED;
      ScaleRows& o = g.a[g.n];
      o.Q = (const bf16*)a.Q; o.ldq = a.ldq; o.z = a.z; o.Qz = (bf16*)a.Qz; o.ldqz = a.ldqz; o.rows = (int)a.r; o.cols = (int)a.d_in;
      if (o.cols > 0) max_units = std::max<int64_t>(max_units, o.rows);
    }
    if (max_units <= 0) continue;
    const int gx = (int)std::min<int64_t>((max_units + kScaleRows - 1) / kScaleRows, 1024);
    launch_k(scale_rows_group_kernel, dim3((unsigned)gx, (unsigned)g.n), dim3(256), (size_t)0, st, g);
    count_launch();
    FLOP_CUDA(cudaGetLastError());
  }
  return FLOP_OK;
}

int flop_active_ranks_gather(const flop_active_gather_t* pr, int n, int dt, void* stream) {
  if (n < 0 || (n > 0 && !pr)) return FLOP_ERR_INVALID_ARG;
  if (dt != FLOP_BF16) return FLOP_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  for (int i0 = 0; i0 < n; i0 += kActiveGroup) {
    ActiveGatherGroup g;
    memset(&g, 0, sizeof(g));
    int max_blocks = 0, max_r = 0;
    for (; g.n < kActiveGroup && i0 + g.n < n; ++g.n) {
      const flop_active_gather_t& a = pr[i0 + g.n];
      if (a.r <= 0 || a.d_in <= 0 || a.d_out <= 0 || a.r > INT32_MAX / 2 || a.d_in > INT32_MAX || a.d_out > INT32_MAX / 2)
        return FLOP_ERR_INVALID_ARG;
      if (!a.z || !a.P || !a.Q || !a.idx || !a.pos || !a.k_dev || !a.z_c || !a.P_c || !a.Q_c || a.ldp < a.r || a.ldq < a.d_in ||
          a.ldpc < a.r || a.ldqc < a.d_in || (a.dz_dla_c && !a.dz_dla) || (a.Qz_c && a.ldqzc < a.d_in))
        return FLOP_ERR_INVALID_ARG;
      if (!bf16_ok(a.P, a.ldp) || !bf16_ok(a.Q, a.ldq) || !bf16_ok(a.P_c, a.ldpc) || !bf16_ok(a.Q_c, a.ldqc) ||
          (a.Qz_c && !bf16_ok(a.Qz_c, a.ldqzc)))
        return FLOP_ERR_UNSUPPORTED;
      if ((size_t)a.r * 2 * kActiveWarps > (size_t)kSmemBudget) return FLOP_ERR_UNSUPPORTED;
      ActiveGather& o = g.a[g.n];
      o.z = a.z; o.dz_dla = a.dz_dla; o.P = (const bf16*)a.P; o.ldp = a.ldp; o.Q = (const bf16*)a.Q; o.ldq = a.ldq;
      o.r = (int)a.r; o.d_in = (int)a.d_in; o.d_out = (int)a.d_out; o.idx = a.idx; o.pos = a.pos; o.k_dev = a.k_dev;
      o.z_c = a.z_c; o.dz_dla_c = a.dz_dla_c; o.P_c = (bf16*)a.P_c; o.ldpc = a.ldpc; o.Q_c = (bf16*)a.Q_c; o.ldqc = a.ldqc;
      o.Qz_c = (bf16*)a.Qz_c; o.ldqzc = a.ldqzc;
      max_blocks = std::max(max_blocks, o.r + o.d_out);
      max_r = std::max(max_r, o.r);
    }
    launch_k(active_select_kernel, dim3(g.n), dim3(1024), (size_t)0, st, g);
    const int row_elems = (max_r + 7) & ~7;   // per-warp staging row, 16-byte aligned
    const size_t smem = (size_t)row_elems * 2 * kActiveWarps;
    if (smem > 48 * 1024) FLOP_CUDA(cudaFuncSetAttribute(active_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    launch_k(active_gather_kernel, dim3((max_blocks + kActiveWarps - 1) / kActiveWarps, g.n), dim3(32 * kActiveWarps), smem, st, g, row_elems);
    count_launch(2);
    FLOP_CUDA(cudaGetLastError());
  }
  return FLOP_OK;
}

int flop_active_ranks_scatter(const flop_active_scatter_t* pr, int n, int accumulate, int wgrad_dt, void* stream) {
  if (n < 0 || (n > 0 && !pr) || !valid_dt(wgrad_dt)) return FLOP_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  for (int i0 = 0; i0 < n; i0 += kActiveGroup) {
    ActiveScatterGroup g;
    memset(&g, 0, sizeof(g));
    g.accumulate = accumulate;
    int max_blocks = 0;
    for (; g.n < kActiveGroup && i0 + g.n < n; ++g.n) {
      const flop_active_scatter_t& a = pr[i0 + g.n];
      if (a.r <= 0 || a.d_in <= 0 || a.d_out <= 0 || a.r > INT32_MAX / 2 || a.d_in > INT32_MAX || a.d_out > INT32_MAX / 2 || !a.idx ||
          !a.pos || !a.k_dev)
        return FLOP_ERR_INVALID_ARG;
      if ((a.dP && (!a.dP_c || a.lddp < a.r || a.lddpc < a.r)) || (a.dQ && (!a.dQ_c || a.lddq < a.d_in || a.lddqc < a.d_in)) ||
          (a.dlog_alpha && !a.dlog_alpha_c))
        return FLOP_ERR_INVALID_ARG;
      ActiveScatter& o = g.a[g.n];
      o.idx = a.idx; o.pos = a.pos; o.k_dev = a.k_dev; o.r = (int)a.r; o.d_in = (int)a.d_in; o.d_out = (int)a.d_out;
      o.dP_c = a.dP_c; o.lddpc = a.lddpc; o.dQ_c = a.dQ_c; o.lddqc = a.lddqc; o.dla_c = a.dlog_alpha_c;
      o.dP = a.dP; o.lddp = a.lddp; o.dQ = a.dQ; o.lddq = a.lddq; o.dla = a.dlog_alpha;
      max_blocks = std::max(max_blocks, o.r + o.d_out);
    }
    if (wgrad_dt == FLOP_BF16) launch_k(active_scatter_kernel<bf16>, dim3((max_blocks + kActiveWarps - 1) / kActiveWarps, g.n), dim3(32 * kActiveWarps), (size_t)0, st, g);
    else                       launch_k(active_scatter_kernel<float>, dim3((max_blocks + kActiveWarps - 1) / kActiveWarps, g.n), dim3(32 * kActiveWarps), (size_t)0, st, g);
    count_launch();
    FLOP_CUDA(cudaGetLastError());
  }
  return FLOP_OK;
}

int flop_expected_l0_lagrangian(const float* log_alpha, int64_t n, const int64_t* seg_off, const float* seg_size,
                                int32_t n_seg, flop_hc_params_t hc, const float* target, const float* lambda,
                                float* out4, float* seg_expected, float* dlog_alpha, void* ws, size_t ws_bytes,
                                void* stream) {
  if (n < 0 || n_seg < 0 || !valid_hc(hc) || !out4 || !target || !lambda) return FLOP_ERR_INVALID_ARG;
  if (n_seg > kL0MaxSeg) return FLOP_ERR_UNSUPPORTED;
  if (n_seg > 0 && (!seg_off || !seg_size)) return FLOP_ERR_INVALID_ARG;
  if (n > 0 && !log_alpha) return FLOP_ERR_INVALID_ARG;
  const size_t need = l0_ws_bytes(n, n_seg);
  FLOP_TRY(check_ws(ws, ws_bytes, need));
  cudaStream_t st = (cudaStream_t)stream;
  L0Scratch* sc = (L0Scratch*)ws;
  const float thr = (float)((double)hc.beta * log(-(double)hc.gamma / (double)hc.zeta));
  const int64_t chunks = (n + kL0Chunk - 1) / kL0Chunk + n_seg;
  if (chunks > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  if (chunks > 0 && n_seg > 0) {
    launch_k(l0_chunk_kernel<false>, dim3((unsigned)chunks), dim3(kL0Threads), (size_t)(0), st, log_alpha, seg_off, seg_size, n_seg, thr, sc, nullptr, n, (int)chunks);
    count_launch();
  }
  launch_k(l0_finalize_kernel, dim3(1), dim3(kL0Threads), (size_t)(0), st, seg_off, seg_size, n_seg, target, lambda, sc, out4, seg_expected, n, (int)chunks);
  count_launch();
  if (dlog_alpha && chunks > 0 && n_seg > 0) {
    launch_k(l0_chunk_kernel<true>, dim3((unsigned)chunks), dim3(kL0Threads), (size_t)(0), st, log_alpha, seg_off, seg_size, n_seg, thr, sc, dlog_alpha, n, (int)chunks);
    count_launch();
  }
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

int flop_expected_l0_lagrangian_noalloc(const float* log_alpha, int64_t n, const int64_t* seg_off,
                                        const float* seg_size, int32_t n_seg, flop_hc_params_t hc,
                                        const float* target, const float* lambda, float* out4,
                                        float* seg_expected, float* dlog_alpha, void* stream) {
  if (n < 0 || n_seg < 0 || !valid_hc(hc) || !out4 || !target || !lambda) return FLOP_ERR_INVALID_ARG;
  if (n > kNoAllocMaxGates || n_seg > kNoAllocMaxSeg) {
    if (debug_on())
      fprintf(stderr, "[flop] flop_expected_l0_lagrangian_noalloc: n=%lld gates / n_seg=%d segments exceed the built-in "
                      "scratch (at most %lld gates, %d segments); use flop_expected_l0_lagrangian with a workspace\n",
              (long long)n, (int)n_seg, (long long)kNoAllocMaxGates, kNoAllocMaxSeg);
    return FLOP_ERR_UNSUPPORTED;
  }
  if (n_seg > 0 && (!seg_off || !seg_size)) return FLOP_ERR_INVALID_ARG;
  if (n > 0 && !log_alpha) return FLOP_ERR_INVALID_ARG;
  L0Scratch* sc = nullptr;
  FLOP_TRY(builtin_scratch(&sc));
  cudaStream_t st = (cudaStream_t)stream;
  const float thr = (float)((double)hc.beta * log(-(double)hc.gamma / (double)hc.zeta));
  const int64_t chunks = (n + kL0Chunk - 1) / kL0Chunk + n_seg;
  // Nothing in the scratch has to start at zero: every chunk sum that the finalisation reads and
  // the gradient coefficient are rewritten by this call before they are read.
  if (chunks > 0 && n_seg > 0) {
    launch_k(l0_chunk_kernel<false>, dim3((unsigned)chunks), dim3(kL0Threads), (size_t)(0), st, log_alpha, seg_off, seg_size, n_seg, thr, sc, nullptr, n, (int)chunks);
    count_launch();
  }
  // the grid, and so the chunk sums this call may use, is sized from the host's n and n_seg; it never exceeds the built-in array
  launch_k(l0_finalize_kernel, dim3(1), dim3(kL0Threads), (size_t)(0), st, seg_off, seg_size, n_seg, target, lambda, sc, out4, seg_expected, n, (int)chunks);
  count_launch();
  if (dlog_alpha && chunks > 0 && n_seg > 0) {
    launch_k(l0_chunk_kernel<true>, dim3((unsigned)chunks), dim3(kL0Threads), (size_t)(0), st, log_alpha, seg_off, seg_size, n_seg, thr, sc, dlog_alpha, n, (int)chunks);
    count_launch();
  }
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

int flop_agp_gates(const float* g, int64_t n, const int64_t* seg_off, int32_t n_seg, const float* sparsity, float l1,
                   float* z, uint8_t* mask, float* dz_dg, float* seg_l1, float* dg, void* stream) {
  if (n < 0 || n_seg < 0 || !sparsity) return FLOP_ERR_INVALID_ARG;
  if (n_seg == 0 || n == 0) return FLOP_OK;
  if (!g || !seg_off || !z) return FLOP_ERR_INVALID_ARG;
  launch_k(agp_gates_kernel, dim3((unsigned)n_seg), dim3(kAgpThreads), (size_t)0, (cudaStream_t)stream, g, seg_off, sparsity, l1, z,
           mask, dz_dg, seg_l1, dg);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  return FLOP_OK;
}

// ---- gated adaptive embedding of one word cluster (Section 4.2): Y = (E[ids] * z) O
static size_t embedding_ws_bytes(int64_t T, int64_t d_i) {
  Arena ar{nullptr, 0, 0};
  ar.take((size_t)T * round_up(std::max<int64_t>(d_i, 1), 8) * 2);                                   // dH'
  const int64_t blocks = (T + kEmbWarps * kEmbTokensPerWarp - 1) / (kEmbWarps * kEmbTokensPerWarp);
  ar.take((size_t)std::max<int64_t>(blocks, 1) * std::max<int64_t>(d_i, 1) * 4);                     // dz partials
  return align_up(ar.used, 256);
}

int flop_gated_embedding_fwd(const int32_t* ids, int64_t T, const void* E, int64_t lde, int64_t n_rows, const void* O,
                             int64_t ldo, const float* z, void* Y, int64_t ldy, void* H_save, int64_t ldh, int64_t d_i,
                             int64_t d, int dt, void* stream) {
  if (T < 0 || n_rows < 0 || d_i < 0 || d < 0 || !valid_dt(dt)) return FLOP_ERR_INVALID_ARG;
  if (dt != FLOP_BF16) return FLOP_ERR_UNSUPPORTED;
  if (T == 0 || d == 0) return FLOP_OK;
  if (d_i == 0 || n_rows == 0) return bf16_ok(Y, ldy) ? zero_2d<bf16>(Y, ldy, T, d, (cudaStream_t)stream) : FLOP_ERR_UNSUPPORTED;
  if (!ids || !z || !check_mat(E, lde, d_i) || !check_mat(O, ldo, d) || !check_mat(Y, ldy, d) || !check_mat(H_save, ldh, d_i))
    return FLOP_ERR_INVALID_ARG;
  if (!bf16_ok(E, lde) || !bf16_ok(O, ldo) || !bf16_ok(Y, ldy) || !bf16_ok(H_save, ldh)) return FLOP_ERR_UNSUPPORTED;
  if (T > INT32_MAX || n_rows > INT32_MAX || d_i > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  launch_k(embed_gather_kernel, dim3((unsigned)((T + kEmbWarps - 1) / kEmbWarps)), dim3(32 * kEmbWarps), (size_t)0, st, ids, (int)T,
           (const bf16*)E, lde, (int)n_rows, z, (int)d_i, (bf16*)H_save, ldh);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  // Y[T, d] = H'[T, d_i] O[d_i, d]: B(n, k) = O[k, n] is read "transposed" (MN-major)
  const TcPlan pl = plan_tc(T, d, d_i, false, true);
  return launch_tc({H_save, ldh, false}, {O, ldo, true}, T, d, d_i, pl, store_epilogue(Y, ldy, nullptr), st);
}

int flop_gated_embedding_bwd(const void* dY, int64_t lddy, const int32_t* ids, int64_t T, const void* E, int64_t lde,
                             int64_t n_rows, const void* O, int64_t ldo, const float* z, const float* dz_dla,
                             const void* H_save, int64_t ldh, float* dE, int64_t ldde, void* dO, int64_t lddo,
                             float* dlog_alpha, int accumulate, int64_t d_i, int64_t d, int dt, int wgrad_dt, void* ws,
                             size_t ws_bytes, void* stream) {
  if (T < 0 || n_rows < 0 || d_i < 0 || d < 0 || !valid_dt(dt) || !valid_dt(wgrad_dt)) return FLOP_ERR_INVALID_ARG;
  if (dt != FLOP_BF16) return FLOP_ERR_UNSUPPORTED;
  if ((dE && ldde < d_i) || (dO && lddo < d) || (dlog_alpha && !dz_dla)) return FLOP_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (T == 0 || d == 0 || d_i == 0 || n_rows == 0) {      // empty batch or empty cluster: gradients are zero
    if (!accumulate) {
      if (dO) FLOP_TRY(wgrad_dt == FLOP_BF16 ? zero_2d<bf16>(dO, lddo, d_i, d, st) : zero_2d<float>(dO, lddo, d_i, d, st));
      if (dlog_alpha) FLOP_TRY(zero_2d<float>(dlog_alpha, d_i, 1, d_i, st));
    }
    return FLOP_OK;
  }
  if (!ids || !z || !check_mat(dY, lddy, d) || !check_mat(E, lde, d_i) || !check_mat(O, ldo, d) || !check_mat(H_save, ldh, d_i))
    return FLOP_ERR_INVALID_ARG;
  if (!bf16_ok(dY, lddy) || !bf16_ok(E, lde) || !bf16_ok(O, ldo) || !bf16_ok(H_save, ldh)) return FLOP_ERR_UNSUPPORTED;
  if (T > INT32_MAX || n_rows > INT32_MAX || d_i > INT32_MAX) return FLOP_ERR_UNSUPPORTED;
  if ((size_t)kEmbWarps * d_i * 4 > (size_t)kSmemBudget) return FLOP_ERR_UNSUPPORTED;
  if (dO && !wgrad_direct_ok(dO, lddo, wgrad_dt)) return FLOP_ERR_UNSUPPORTED;   // dO is written in place with 16-byte stores
  FLOP_TRY(check_ws(ws, ws_bytes, embedding_ws_bytes(T, d_i)));
  Arena ar{(unsigned char*)ws, ws_bytes, 0};
  const int64_t lddh = round_up(d_i, 8);
  bf16* dH = (bf16*)ar.take((size_t)T * lddh * 2);
  const int64_t blocks = (T + kEmbWarps * kEmbTokensPerWarp - 1) / (kEmbWarps * kEmbTokensPerWarp);
  float* part = (float*)ar.take((size_t)blocks * d_i * 4);
  // dH'[T, d_i] = dY[T, d] O^T: B(n = k_dim, k = j) = O[n, j] (K-major as stored)
  FLOP_TRY(launch_tc({dY, lddy, false}, {O, ldo, false}, T, d_i, d, plan_tc(T, d_i, d, false, false),
                     store_epilogue(dH, lddh, nullptr), st));
  if (dO) {
    // dO[d_i, d] = H'^T dY: contraction over tokens, written in place when the output allows 16-byte vectors
    TcPlan pl = plan_tc(d_i, d, T, false, true);
    FLOP_TRY(launch_tc({H_save, ldh, true}, {dY, lddy, true}, d_i, d, T, pl, wgrad_epilogue(dO, lddo, wgrad_dt, nullptr, accumulate), st));
  }
  if (dE || dlog_alpha) {
    const size_t smem = (size_t)kEmbWarps * d_i * 4;
    if (smem > 48 * 1024) FLOP_CUDA(cudaFuncSetAttribute(embed_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    launch_k(embed_bwd_kernel, dim3((unsigned)blocks), dim3(32 * kEmbWarps), smem, st, ids, (int)T, (const bf16*)E, lde, (int)n_rows, z,
             (int)d_i, (const bf16*)dH, lddh, dE, ldde, dlog_alpha ? part : nullptr);
    count_launch();
    if (dlog_alpha) {
      launch_k(dalpha_kernel, dim3((unsigned)((d_i + 255) / 256)), dim3(256), (size_t)0, st, (const float*)part, (int)blocks, d_i, dz_dla,
               (int)d_i, dlog_alpha, accumulate);
      count_launch();
    }
    FLOP_CUDA(cudaGetLastError());
  }
  return FLOP_OK;
}

int flop_compact_ranks(const float* log_alpha_or_z, int mode, flop_hc_params_t hc, int64_t r, const void* P, int64_t ldp,
                       const void* Q, int64_t ldq, int64_t d_in, int64_t d_out, int dt, int32_t* idx, int32_t* k_dev,
                       float* z_det, void* Pc, int64_t ldpc, void* Qc, int64_t ldqc, void* ws, size_t ws_bytes,
                       void* stream) {
  (void)ws; (void)ws_bytes;
  if (r < 0 || d_in < 0 || d_out < 0 || (mode != 0 && mode != 1) || !valid_dt(dt) || !k_dev) return FLOP_ERR_INVALID_ARG;
  if (mode == 0 && !valid_hc(hc)) return FLOP_ERR_INVALID_ARG;
  if (r > 65536) return FLOP_ERR_UNSUPPORTED;
  if (r > 0 && (!log_alpha_or_z || !idx)) return FLOP_ERR_INVALID_ARG;
  const bool gather = P || Q || Pc || Qc;
  if (gather) {
    if (!P || !Q || !Pc || !Qc || ldp < r || ldq < d_in || ldqc < d_in) return FLOP_ERR_INVALID_ARG;
    if (!z_det && mode == 0) return FLOP_ERR_INVALID_ARG;   // the gather scales Q rows by the deterministic gate
  }
  cudaStream_t st = (cudaStream_t)stream;
  const double thr = (double)hc.beta * log(-(double)hc.gamma / (double)hc.zeta);
  launch_k(compact_select_kernel, dim3(1), dim3(kSelThreads), (size_t)(0), st, log_alpha_or_z, mode, thr, (int)r, idx, k_dev, z_det);
  count_launch();
  FLOP_CUDA(cudaGetLastError());
  if (gather && r > 0) {
    const float* zsrc = z_det ? z_det : log_alpha_or_z;
    const size_t es = elt(dt);
    const int vq = aligned16(Q) && aligned16(Qc) && (ldq * es) % 16 == 0 && (ldqc * es) % 16 == 0;
    const int vp = aligned16(P) && (ldp * es) % 16 == 0;
    const int rows_per_block = 1;   // one P row per block: many resident blocks overlap one row's load with another's gather
    const size_t smem = (size_t)r * es;
    if (smem > (size_t)kSmemBudget) return FLOP_ERR_UNSUPPORTED;
    if (dt == FLOP_BF16) {
      if (d_in > 0) launch_k(gather_q_kernel<bf16>, dim3((unsigned)r), dim3(256), (size_t)(0), st, (const bf16*)Q, ldq, idx, k_dev, zsrc, (int)d_in, (bf16*)Qc, ldqc, vq);
      // rows staged by bulk asynchronous copies when they are 16-byte pieces
      const int pipe_on = tuning().gather_pipe;
      if (d_out > 0 && pipe_on && vp && r % 8 == 0) {
        const size_t row_bytes = (size_t)r * 2, idx_bytes = (row_bytes + 127) & ~(size_t)127;
        int rows_per_stage = (int)std::max<size_t>(1, std::min<size_t>(16, (16 * 1024) / row_bytes));
        int nbuf = kGatherMaxBuf;
        auto need = [&](int nb) { return 64 + idx_bytes + (size_t)nb * rows_per_stage * row_bytes; };
        while (nbuf > 2 && need(nbuf) > 100 * 1024) --nbuf;   // two blocks per SM where the rows allow it
        if (need(nbuf) <= (size_t)kSmemBudget) {
          const size_t sm = need(nbuf);
          static bool configured[kMaxDevices] = {};
          if (sm > 48 * 1024 && first_use_on_device(configured))
            FLOP_CUDA(cudaFuncSetAttribute(gather_p_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget));
          const int64_t groups = (d_out + rows_per_stage - 1) / rows_per_stage;
          const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(8, (size_t)(224 * 1024) / sm));
          const int grid = (int)std::min<int64_t>(groups, (int64_t)num_sms() * per_sm);
          launch_k(gather_p_pipe_kernel, dim3((unsigned)grid), dim3(256), sm, st, (const bf16*)P, ldp, idx, k_dev, (int)r, (int)d_out,
                   (bf16*)Pc, ldpc, rows_per_stage, nbuf);
        } else {
          if (smem > 48 * 1024) FLOP_CUDA(cudaFuncSetAttribute(gather_p_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
          launch_k(gather_p_kernel<bf16>, dim3((unsigned)((d_out + rows_per_block - 1) / rows_per_block)), dim3(256), (size_t)(smem), st,
              (const bf16*)P, ldp, idx, k_dev, (int)r, (int)d_out, (bf16*)Pc, ldpc, rows_per_block, vp);
        }
      } else if (d_out > 0) {
        if (smem > 48 * 1024) FLOP_CUDA(cudaFuncSetAttribute(gather_p_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        launch_k(gather_p_kernel<bf16>, dim3((unsigned)((d_out + rows_per_block - 1) / rows_per_block)), dim3(256), (size_t)(smem), st, 
            (const bf16*)P, ldp, idx, k_dev, (int)r, (int)d_out, (bf16*)Pc, ldpc, rows_per_block, vp);
      }
    } else {
      if (d_in > 0) launch_k(gather_q_kernel<float>, dim3((unsigned)r), dim3(256), (size_t)(0), st, (const float*)Q, ldq, idx, k_dev, zsrc, (int)d_in, (float*)Qc, ldqc, vq);
      if (d_out > 0) {
        if (smem > 48 * 1024) FLOP_CUDA(cudaFuncSetAttribute(gather_p_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        launch_k(gather_p_kernel<float>, dim3((unsigned)((d_out + rows_per_block - 1) / rows_per_block)), dim3(256), (size_t)(smem), st, 
            (const float*)P, ldp, idx, k_dev, (int)r, (int)d_out, (float*)Pc, ldpc, rows_per_block, vp);
      }
    }
    count_launch((d_in > 0) + (d_out > 0));
    FLOP_CUDA(cudaGetLastError());
  }
  return FLOP_OK;
}

}  // extern "C"

// C ABI of the verification library (declared in include/pyramidsd.h): argument validation, scratch
// management and kernel launches. No torch types, no CPU fallback: every step of the path runs in the
// kernels of this directory.
#include "../../include/pyramidsd.h"
#include "../../include/pyramidsd_diag.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "finalize.cuh"
#include "rowstats_baseline.cuh"
#include "rowstats_cluster.cuh"
#include "rowstats_onepass.cuh"
#include "lmhead_fused.cuh"

namespace {

using psd::RowStats;
using psd::StageParams;

std::atomic<uint64_t> g_launches{0};
thread_local cudaStream_t t_stream = nullptr;
thread_local int t_two_stage_policy = PSD_TWO_STAGE_AUTO;

constexpr int kMaxDevices = 64;
constexpr size_t kAlign = 256;

// Scratch of pyramidsd_verify_stage_noalloc: per-row statistics for up to PSD_NOALLOC_MAX_ROWS rows, then one
// 256-byte line whose first word is the wait-timeout flag. It is part of the library image, so every
// device that loads the library carries it until the process ends. In host code this name is only a
// handle for cudaGetSymbolAddress; the device address it yields is what kernels are given.
constexpr size_t kNoAllocStatsBytes = static_cast<size_t>(PSD_NOALLOC_MAX_ROWS) * sizeof(RowStats);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocStatsBytes + kAlign];
void* g_noalloc_ptr[kMaxDevices] = {};
std::mutex g_noalloc_mu;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Library-owned scratch. Every (device, stream) pair that has been used without a caller workspace owns its own
// buffers: the workspace of the stage / pyramid calls, the status word of the bounded waits, the staging
// buffers of the host-pointer entry point and the partial sums of the fused LM-head. A call touches only the
// buffers of the stream it runs on and holds that entry's mutex while it enqueues, so two host threads on two
// streams share nothing and two threads on one stream take turns. Buffers are grown on demand (after waiting
// for the stream's own earlier work, which is all that can still use them), never shrunk, and freed at
// process exit by the driver.
struct StreamScratch {
  std::mutex mu;
  bool used = false;
  cudaStream_t stream = nullptr;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int* status = nullptr;
  void* stage[4] = {nullptr, nullptr, nullptr, nullptr};
  size_t stage_bytes[4] = {0, 0, 0, 0};
  void* out4 = nullptr;     // 4 x [B] results of the host entry point
  size_t out4_bytes = 0;
  void* lm_ws = nullptr;    // partial sums of the fused LM-head path
  size_t lm_ws_bytes = 0;
  void* draw = nullptr;     // records and tile totals of the three-launch finalisation
  size_t draw_bytes = 0;
};
struct DeviceState {
  std::mutex mu;
  StreamScratch streams[PSD_MAX_STREAMS];
  // PSD_TWO_STAGE_AUTO: window lengths of a recent call, written by the stage-1 finalisation straight into
  // mapped host memory (a hint for the schedule only: racing writers cannot change any result)
  int32_t* fill_host = nullptr;
  int32_t* fill_dev = nullptr;
  int fill_B = 0, fill_Kq = 0;   // the shape those lengths belong to
  unsigned fill_calls = 0;       // calls of that shape since the lengths were last asked for
};
constexpr int kFillCap = 4096;
DeviceState g_dev[kMaxDevices];
// what pyramidsd_last_status() looks at: the stream and the status word of this thread's most recent call (the word
// sits in a scratch entry, or in the tail of the caller's workspace)
thread_local StreamScratch* t_last_scratch = nullptr;
thread_local int* t_last_status = nullptr;
thread_local cudaStream_t t_last_stream = nullptr;

int current_device_state(DeviceState** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSD_ERR_CUDA;
  *out = &g_dev[dev];
  return PSD_OK;
}

// The scratch entry of `stream` on the current device, created on first use; its status word exists on return.
int scratch_for(cudaStream_t stream, StreamScratch** out) {
  DeviceState* ds = nullptr;
  int rc = current_device_state(&ds);
  if (rc != PSD_OK) return rc;
  StreamScratch* ss = nullptr;
  {
    std::lock_guard<std::mutex> lock(ds->mu);
    for (auto& e : ds->streams)
      if (e.used && e.stream == stream) { ss = &e; break; }
    if (ss == nullptr)
      for (auto& e : ds->streams)
        if (!e.used) { e.used = true; e.stream = stream; ss = &e; break; }
  }
  if (ss == nullptr) {
    std::fprintf(stderr, "pyramidsd: more than %d streams in use on this device; supply a workspace\n", PSD_MAX_STREAMS);
    return PSD_ERR_WORKSPACE;
  }
  *out = ss;
  return PSD_OK;
}

// with ss->mu held
int ensure_status(StreamScratch* ss) {
  if (ss->status) return PSD_OK;
  if (cudaMalloc(reinterpret_cast<void**>(&ss->status), kAlign) != cudaSuccess) { cudaGetLastError(); return PSD_ERR_CUDA; }
  if (cudaMemset(ss->status, 0, kAlign) != cudaSuccess) return PSD_ERR_CUDA;
  return PSD_OK;
}

// with ss->mu held: only work already enqueued on ss->stream can still use the old buffer
int grow(StreamScratch* ss, void** ptr, size_t* have, size_t want) {
  if (*have >= want) return PSD_OK;
  if (*ptr) {
    if (cudaStreamSynchronize(ss->stream) != cudaSuccess) return PSD_ERR_CUDA;
    cudaFree(*ptr);
    *ptr = nullptr;
    *have = 0;
  }
  if (cudaMalloc(ptr, want) != cudaSuccess) { cudaGetLastError(); return PSD_ERR_CUDA; }
  *have = want;
  return PSD_OK;
}

size_t stats_bytes(long long rows) { return align_up(static_cast<size_t>(rows) * sizeof(RowStats)); }

size_t stage_workspace_bytes(int B, int K) {
  // per-row statistics, a [B, K] window and a [B] length (the last two are used by the wrapper only)
  return stats_bytes(static_cast<long long>(B) * K) + align_up(static_cast<size_t>(B) * K * 4) +
         align_up(static_cast<size_t>(B) * 4) + kAlign;
}

bool valid_dtype(int d) { return d == PSD_F32 || d == PSD_BF16; }
bool valid_mode(int m) { return m >= PSD_FUZZY && m <= PSD_ASSISTED; }
bool valid_div(int d) { return d >= PSD_DIV_JS && d <= PSD_DIV_KL; }
size_t elem_size(int dtype) { return dtype == PSD_F32 ? 4 : 2; }

constexpr int kMaxV = psd::kFinTile * psd::kFinMaxTiles;

__global__ void row_uniforms_kernel(unsigned long long seed, unsigned long long offset, int n_rows, float* out_u,
                                    float* out_u2) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= n_rows) return;
  float u, u2;
  psd::row_uniforms(seed, offset, static_cast<unsigned>(r), &u, &u2);
  if (out_u) out_u[r] = u;
  if (out_u2) out_u2[r] = u2;
}

// Optional event bracketing of each launch (pyramidsd_kernel_timing_begin/_end).
constexpr int kMaxTimed = 4096;
struct Timing {
  bool on = false;
  int n = 0;
  cudaEvent_t ev[kMaxTimed][2];
  int created = 0;
  int tag[kMaxTimed];
};
thread_local Timing t_timing;

struct TimedLaunch {
  cudaStream_t s;
  int slot = -1;
  TimedLaunch(cudaStream_t stream, int tag) : s(stream) {
    Timing& t = t_timing;
    if (!t.on || t.n >= kMaxTimed) return;
    if (t.n >= t.created) {
      if (cudaEventCreate(&t.ev[t.n][0]) != cudaSuccess || cudaEventCreate(&t.ev[t.n][1]) != cudaSuccess) return;
      t.created = t.n + 1;
    }
    slot = t.n++;
    t.tag[slot] = tag;
    cudaEventRecord(t.ev[slot][0], s);
  }
  ~TimedLaunch() {
    if (slot >= 0) cudaEventRecord(t_timing.ev[slot][1], s);
  }
};

int check_launch() {
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    std::fprintf(stderr, "pyramidsd: kernel launch failed: %s\n", cudaGetErrorString(e));
    return PSD_ERR_CUDA;
  }
  return PSD_OK;
}

// Statistics pass for one stage: picks the kernel variant and launches it. `allow_triples`: a wrapper launch may
// walk its rows as (draft, qualifier, target) triples where the geometry streams them twice. `resid_wanted`: some
// caller output takes the rows' residual masses (without them the KL divergence goes through the one-pass kernel).
// `onepass`: 1 / 0 = the caller has decided for / against the one-pass kernel (a two-stage call decides once, on its
// whole shape, so that all its schedules run the same arithmetic); -1 = decide here.
int launch_rowstats(const StageParams& P, int dtype, int variant, int cluster_size, cudaStream_t stream,
                    bool allow_triples = false, bool resid_wanted = true, int onepass = -1) {
  const long long rows = static_cast<long long>(P.B) * P.K;
  if (rows == 0 && P.K2 == 0) return PSD_OK;
  if (onepass < 0) onepass = (variant == PSD_KERNEL_AUTO && cluster_size == 0 && psd::onepass_applies(P, dtype, resid_wanted)) ? 1 : 0;
  if (onepass == 1) {
    TimedLaunch timed(stream, 0);
    if (psd::launch_rowstats_onepass(P, dtype, stream, allow_triples) != 0) {
      const cudaError_t e = cudaGetLastError();
      std::fprintf(stderr, "pyramidsd: one-pass kernel launch failed: %s\n", cudaGetErrorString(e));
      return PSD_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return check_launch();
  }
  bool use_cluster = false;
  psd::ClusterGeom geom{};
  if (variant != PSD_KERNEL_BASELINE) {
    use_cluster = psd::cluster_geometry(P, dtype, cluster_size, variant == PSD_KERNEL_CLUSTER_STREAMED, allow_triples, &geom);
    if (!use_cluster && variant != PSD_KERNEL_AUTO) return PSD_ERR_UNSUPPORTED;
  }
  TimedLaunch timed(stream, 0);
  if (use_cluster) {
    if (psd::launch_rowstats_cluster(P, dtype, geom, stream) != 0) {
      const cudaError_t e = cudaGetLastError();
      std::fprintf(stderr, "pyramidsd: cluster kernel launch failed: %s\n", cudaGetErrorString(e));
      return PSD_ERR_CUDA;
    }
  } else {
    const dim3 block(1024);
    if (rows > 0) {
      const dim3 grid(static_cast<unsigned>(rows));
      if (dtype == PSD_F32) psd::rowstats_baseline_kernel<float><<<grid, block, 0, stream>>>(P);
      else psd::rowstats_baseline_kernel<__nv_bfloat16><<<grid, block, 0, stream>>>(P);
    }
    if (P.K2 > 0) {   // the second row set as a launch of its own
      StageParams Q = P;
      Q.small = P.small2; Q.large = P.large2;
      Q.seq_stride_small = P.seq_stride_small2; Q.seq_stride_large = P.seq_stride_large2;
      Q.K = P.K2; Q.K2 = 0; Q.stats = P.stats2; Q.n_valid = nullptr;
      const dim3 grid(static_cast<unsigned>(static_cast<long long>(P.B) * P.K2));
      if (dtype == PSD_F32) psd::rowstats_baseline_kernel<float><<<grid, block, 0, stream>>>(Q);
      else psd::rowstats_baseline_kernel<__nv_bfloat16><<<grid, block, 0, stream>>>(Q);
      g_launches.fetch_add(1, std::memory_order_relaxed);
    }
  }
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return check_launch();
}

// The finalisation kernels run as clusters of CL CTAs per sequence (per stage in the split form): four while
// that still leaves SMs to spare, fewer for large batches, where one CTA per sequence already fills the GPU.
template <typename Kernel, typename... Args>
cudaError_t launch_fin_clusters(Kernel kernel, int cl, unsigned units, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(units * static_cast<unsigned>(cl));
  cfg.blockDim = dim3(psd::kFinThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = static_cast<unsigned>(cl);
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  // a programmatic dependent of the statistics launch before it: its CTAs may be placed while that launch drains,
  // and wait (griddepcontrol.wait, their first instruction) for its end before they read a statistic
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

int fin_cluster_size(long long units) {
  int sms = psd::cluster_sm_count();
  if (sms <= 0) sms = 148;
  if (units * 4 <= 2ll * sms) return 4;
  if (units * 2 <= 2ll * sms) return 2;
  return 1;
}

#define PSD_FIN_DISPATCH(KERNEL, T, cl, units, stream, ...)                                              \
  ((cl) == 4 ? launch_fin_clusters(psd::KERNEL<T, 4>, 4, units, stream, __VA_ARGS__)                        \
   : (cl) == 2 ? launch_fin_clusters(psd::KERNEL<T, 2>, 2, units, stream, __VA_ARGS__)                      \
               : launch_fin_clusters(psd::KERNEL<T, 1>, 1, units, stream, __VA_ARGS__))

// Whether a finalisation of `units` sequences (x stages) goes as three launches (scan, tile totals, pick): batches of
// 64 and more (measured: below that the one-launch form, four CTAs per sequence, is the faster one), within the
// limits of the draw records.
constexpr long long kSplitMinUnits = 64;
bool split_finalize(long long units, int V, bool bonus, const StreamScratch* ss) {
  if (ss == nullptr || bonus) return false;
  if (units < kSplitMinUnits || units > psd::kDrawMaxUnits) return false;
  return (V + psd::kFinTile - 1) / psd::kFinTile <= psd::kDrawMaxTiles;
}

// A launch that may begin while the launch before it on the stream drains (programmatic dependent launch): the
// kernel itself waits, with griddepcontrol.wait, before it reads what that launch wrote.
template <typename Kernel, typename... Args>
cudaError_t launch_dependent(Kernel kernel, unsigned grid, unsigned block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

int launch_finalize_split(const StageParams& P1, const StageParams& P2, int n_stages, int dtype, cudaStream_t stream,
                        StreamScratch* ss) {
  const long long units = static_cast<long long>(n_stages) * P1.B;
  int rc = grow(ss, &ss->draw, &ss->draw_bytes, psd::draw_scratch_bytes(units));
  if (rc != PSD_OK) return rc;
  psd::DrawScratch d;
  char* base = static_cast<char*>(ss->draw);
  d.tile_total = reinterpret_cast<double*>(base);
  base += static_cast<size_t>(units) * psd::kDrawMaxTiles * sizeof(double);
  d.record = reinterpret_cast<psd::DrawRecord*>(base);
  base += static_cast<size_t>(units) * sizeof(psd::DrawRecord);
  d.drawn = reinterpret_cast<psd::DrawRecord*>(base);
  base += static_cast<size_t>(units) * sizeof(psd::DrawRecord);
  d.need = reinterpret_cast<int*>(base);
  d.count = d.need + units;   // in the 256 spare bytes
  int sms = psd::cluster_sm_count();
  if (sms <= 0) sms = 148;
  const unsigned scan_ctas = static_cast<unsigned>((units + psd::kScanWarps - 1) / psd::kScanWarps);
  TimedLaunch timed(stream, 1);
  if (dtype == PSD_F32) {
    launch_dependent(psd::finalize_scan_kernel<float>, scan_ctas, psd::kScanWarps * 32, stream, P1, P2, n_stages, d);
    launch_dependent(psd::finalize_tiles_kernel<float>, sms, psd::kFinThreads, stream, P1, P2, n_stages, d);
    launch_dependent(psd::finalize_pick_kernel<float>, sms, psd::kFinThreads, stream, P1, P2, n_stages, d);
  } else {
    launch_dependent(psd::finalize_scan_kernel<__nv_bfloat16>, scan_ctas, psd::kScanWarps * 32, stream, P1, P2, n_stages, d);
    launch_dependent(psd::finalize_tiles_kernel<__nv_bfloat16>, sms, psd::kFinThreads, stream, P1, P2, n_stages, d);
    launch_dependent(psd::finalize_pick_kernel<__nv_bfloat16>, sms, psd::kFinThreads, stream, P1, P2, n_stages, d);
  }
  g_launches.fetch_add(3, std::memory_order_relaxed);
  return check_launch();
}

int launch_finalize(const StageParams& P, int dtype, cudaStream_t stream, StreamScratch* ss = nullptr) {
  if (P.B == 0) return PSD_OK;
  if (split_finalize(P.B, P.V, P.bonus != 0, ss)) return launch_finalize_split(P, P, 1, dtype, stream, ss);
  TimedLaunch timed(stream, 1);
  const int cl = fin_cluster_size(P.B);
  const unsigned units = static_cast<unsigned>(P.B);
  cudaError_t e;
  if (dtype == PSD_F32) e = PSD_FIN_DISPATCH(finalize_kernel, float, cl, units, stream, P);
  else e = PSD_FIN_DISPATCH(finalize_kernel, __nv_bfloat16, cl, units, stream, P);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (e != cudaSuccess) { cudaGetLastError(); return PSD_ERR_CUDA; }
  return check_launch();
}

int validate_stage(const psd_stage_args* a) {
  if (a == nullptr || a->struct_size != sizeof(psd_stage_args)) return PSD_ERR_INVALID_ARG;
  if (!valid_dtype(a->dtype) || !valid_mode(a->mode) || !valid_div(a->div_kind)) return PSD_ERR_INVALID_ARG;
  if (a->B < 0 || a->K < 0 || a->K > 32 || a->V < 1) return PSD_ERR_INVALID_ARG;
  if (a->kernel_variant < PSD_KERNEL_AUTO || a->kernel_variant > PSD_KERNEL_CLUSTER_STREAMED || a->cluster_size < 0) return PSD_ERR_INVALID_ARG;
  if (a->kernel_variant == PSD_KERNEL_CLUSTER_STREAMED && a->cluster_size == 0) return PSD_ERR_INVALID_ARG;
  if (a->seq_index_base < 0 || a->reserved0 != 0) return PSD_ERR_INVALID_ARG;
  if (a->V > kMaxV) return PSD_ERR_UNSUPPORTED;
  if (static_cast<long long>(a->B) * a->K > (1ll << 30)) return PSD_ERR_UNSUPPORTED;
  if (a->inv_temperature < 0.f || std::isnan(a->inv_temperature) || std::isinf(a->inv_temperature)) return PSD_ERR_INVALID_ARG;
  if (std::isnan(a->threshold)) return PSD_ERR_INVALID_ARG;
  if (a->seq_stride_small < 0 || a->seq_stride_large < 0) return PSD_ERR_INVALID_ARG;
  if (a->B > 0) {
    if (!a->out_accept_len || !a->out_next_token) return PSD_ERR_INVALID_ARG;
    if (a->K > 0 && (!a->logits_small || !a->logits_large || !a->tokens)) return PSD_ERR_INVALID_ARG;
    const long long min_stride = static_cast<long long>(a->K) * a->V;
    if (a->seq_stride_small != 0 && a->seq_stride_small < min_stride) return PSD_ERR_INVALID_ARG;
    if (a->seq_stride_large != 0 && a->seq_stride_large < min_stride + (a->large_has_bonus_row ? a->V : 0)) return PSD_ERR_INVALID_ARG;
    if (a->large_has_bonus_row && !a->logits_large) return PSD_ERR_INVALID_ARG;
  }
  if (a->large_has_bonus_row != 0 && a->large_has_bonus_row != 1) return PSD_ERR_INVALID_ARG;
  if (a->workspace != nullptr) {
    if ((reinterpret_cast<uintptr_t>(a->workspace) % kAlign) != 0) return PSD_ERR_WORKSPACE;
    if (a->workspace_bytes < stage_workspace_bytes(a->B, a->K)) return PSD_ERR_WORKSPACE;
  }
  return PSD_OK;
}

StageParams make_params(const psd_stage_args* a, void* ws, int* status) {
  StageParams P{};
  P.small = a->logits_small;
  P.large = a->logits_large;
  P.tokens = a->tokens;
  P.n_valid = a->n_valid;
  P.B = a->B; P.K = a->K; P.V = a->V;
  const long long dense = static_cast<long long>(a->K) * a->V;
  P.seq_stride_small = a->seq_stride_small ? a->seq_stride_small : dense;
  P.seq_stride_large = a->seq_stride_large ? a->seq_stride_large : dense + (a->large_has_bonus_row ? a->V : 0);
  P.bonus = a->large_has_bonus_row;
  const double invT = a->inv_temperature > 0.f ? static_cast<double>(a->inv_temperature) : 1.0;
  P.c = static_cast<float>(1.4426950408889634 * invT);
  P.threshold = a->threshold;
  P.mode = a->mode;
  P.div_kind = a->div_kind;
  P.seed = a->philox_seed;
  P.offset = a->philox_offset;
  P.stats = static_cast<RowStats*>(ws);
  P.out_accept_len = a->out_accept_len;
  P.out_next_token = a->out_next_token;
  P.out_div = a->out_div;
  P.out_p_small_tok = a->out_p_small_tok;
  P.out_p_large_tok = a->out_p_large_tok;
  P.out_resid_mass = a->out_resid_mass;
  P.out_row_flags = a->out_row_flags;
  P.window = nullptr;
  P.n_window = nullptr;
  P.K_window = 0;
  P.status = status;
  P.seq_base = a->seq_index_base;
  return P;
}

cudaStream_t pick_stream(const psd_stage_args* a) {
  if (a->stream != nullptr || a->use_stream_field) return static_cast<cudaStream_t>(a->stream);
  return t_stream;
}

// Runs one stage with the scratch entry `ss` (held by the caller); `window_out`/`n_window_out`/`K_window` non-null
// make the finalisation also build the stage-2 window of the wrapper.
int run_stage_locked(const psd_stage_args* a, StreamScratch* ss, int* status, cudaStream_t stream, int32_t* window_out,
                     int32_t* n_window_out, int K_window, int32_t* fill_out = nullptr, int onepass = -1) {
  int rc = PSD_OK;
  void* ws = a->workspace;
  if (ws == nullptr) {
    rc = grow(ss, &ss->ws, &ss->ws_bytes, stage_workspace_bytes(a->B, a->K));
    if (rc != PSD_OK) return rc;
    ws = ss->ws;
  }
  StageParams P = make_params(a, ws, status);
  P.window = window_out;
  P.n_window = n_window_out;
  P.K_window = K_window;
  P.fill_out = fill_out;
  P.fill_cap = kFillCap;
  if (a->K > 0) {
    rc = launch_rowstats(P, a->dtype, a->kernel_variant, a->cluster_size, stream, false, P.out_resid_mass != nullptr, onepass);
    if (rc != PSD_OK) return rc;
  }
  return launch_finalize(P, a->dtype, stream, ss);
}

int run_stage(const psd_stage_args* a) {
  int rc = validate_stage(a);
  if (rc != PSD_OK) return rc;
  if (a->B == 0) return PSD_OK;
  const cudaStream_t stream = pick_stream(a);
  if (a->workspace != nullptr) {
    // the caller's workspace holds everything, the status word in its last 256 bytes: no library buffer, no allocation
    int* status = reinterpret_cast<int*>(static_cast<char*>(a->workspace) + stage_workspace_bytes(a->B, a->K) - kAlign);
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return PSD_ERR_CUDA;
    t_last_scratch = nullptr; t_last_status = status; t_last_stream = stream;
    return run_stage_locked(a, nullptr, status, stream, nullptr, nullptr, 0);
  }
  StreamScratch* ss = nullptr;
  rc = scratch_for(stream, &ss);
  if (rc != PSD_OK) return rc;
  std::lock_guard<std::mutex> lock(ss->mu);
  rc = ensure_status(ss);
  if (rc != PSD_OK) return rc;
  t_last_scratch = ss; t_last_status = ss->status; t_last_stream = stream;
  return run_stage_locked(a, ss, ss->status, stream, nullptr, nullptr, 0);
}

size_t pyramid_workspace_bytes(int B, int K_d, int K_q) { return stage_workspace_bytes(B, K_d) + stage_workspace_bytes(B, K_q); }

int validate_pyramid(const psd_pyramid_args* a) {
  if (a == nullptr || a->struct_size != sizeof(psd_pyramid_args)) return PSD_ERR_INVALID_ARG;
  if (!valid_dtype(a->dtype) || !valid_mode(a->mode_q) || !valid_mode(a->mode_t) || !valid_div(a->div_kind)) return PSD_ERR_INVALID_ARG;
  if (a->K_q < 1 || a->K_d < a->K_q || a->K_d > 32 || a->B < 0 || a->V < 1) return PSD_ERR_INVALID_ARG;
  if (a->schedule < PSD_TWO_STAGE_DEFAULT || a->schedule > PSD_TWO_STAGE_FUSED_ROWS) return PSD_ERR_INVALID_ARG;
  if (a->kernel_variant != PSD_KERNEL_AUTO && a->kernel_variant != PSD_KERNEL_BASELINE) return PSD_ERR_INVALID_ARG;
  if (a->target_has_bonus_row != 0 && a->target_has_bonus_row != 1) return PSD_ERR_INVALID_ARG;
  if (a->seq_index_base < 0) return PSD_ERR_INVALID_ARG;
  if (a->B > 0 && (!a->logits_draft || !a->logits_qual || !a->logits_target || !a->draft_tokens || !a->out_accept_len_q ||
                   !a->out_next_token_q || !a->out_accept_len || !a->out_next_token))
    return PSD_ERR_INVALID_ARG;
  if (a->workspace != nullptr) {
    if ((reinterpret_cast<uintptr_t>(a->workspace) % kAlign) != 0) return PSD_ERR_WORKSPACE;
    if (a->workspace_bytes < pyramid_workspace_bytes(a->B, a->K_d, a->K_q)) return PSD_ERR_WORKSPACE;
  }
  return PSD_OK;
}

// Both stages of the pyramid with the scratch entry `ss` held by the caller.
int verify_two_stage_locked(const psd_pyramid_args* a, StreamScratch* ss, int* status, cudaStream_t stream) {
  const int B = a->B, K_d = a->K_d, K_q = a->K_q, V = a->V, dtype = a->dtype;
  DeviceState* ds = nullptr;
  int rc = current_device_state(&ds);
  if (rc != PSD_OK) return rc;
  // scratch: [stage-1 workspace][stage-2 workspace]; the window and its length live in stage 1's tail unless the
  // caller wants them
  const size_t ws1 = stage_workspace_bytes(B, K_d), ws2 = stage_workspace_bytes(B, K_q);
  char* base = static_cast<char*>(a->workspace);
  if (base == nullptr) {
    rc = grow(ss, &ss->ws, &ss->ws_bytes, ws1 + ws2);
    if (rc != PSD_OK) return rc;
    base = static_cast<char*>(ss->ws);
  }
  int32_t* window = reinterpret_cast<int32_t*>(base + stats_bytes(static_cast<long long>(B) * K_d));
  int32_t* n_window = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(window) + align_up(static_cast<size_t>(B) * K_d * 4));
  if (a->out_window != nullptr) window = a->out_window;
  if (a->out_n_window != nullptr) n_window = a->out_n_window;

  psd_stage_args s1;
  std::memset(&s1, 0, sizeof(s1));
  s1.struct_size = sizeof(s1);
  s1.dtype = dtype;
  s1.logits_small = a->logits_draft;
  s1.logits_large = a->logits_qual;
  s1.tokens = a->draft_tokens;
  s1.B = B; s1.K = K_d; s1.V = V;
  s1.mode = a->mode_q;
  s1.div_kind = a->div_kind;
  s1.inv_temperature = a->inv_temperature;
  s1.threshold = a->tau_q;
  s1.philox_seed = a->philox_seed;
  s1.philox_offset = a->philox_offset;
  s1.seq_index_base = a->seq_index_base;
  s1.out_accept_len = a->out_accept_len_q;
  s1.out_next_token = a->out_next_token_q;
  s1.out_div = a->out_div_q;
  s1.out_resid_mass = a->out_resid_q;
  s1.workspace = base;
  s1.workspace_bytes = ws1;
  s1.kernel_variant = a->kernel_variant;
  psd_stage_args s2 = s1;
  s2.logits_small = a->logits_qual;   // P_MQ takes the place of P_MD in the target comparison (Fig. 1)
  s2.logits_large = a->logits_target;
  s2.seq_stride_small = static_cast<int64_t>(K_d) * V;  // rows 0..K_q-1 of each [K_d, V] qualifier sequence
  s2.seq_stride_large = 0;
  s2.large_has_bonus_row = a->target_has_bonus_row;   // target [B, K_q + 1, V]: its last row per sequence is the bonus row
  s2.tokens = window;
  s2.n_valid = n_window;
  s2.K = K_q;
  s2.mode = a->mode_t;
  s2.threshold = a->tau_t;
  s2.philox_offset = a->philox_offset + 1;
  s2.out_accept_len = a->out_accept_len;
  s2.out_next_token = a->out_next_token;
  s2.out_div = a->out_div_t;
  s2.out_resid_mass = a->out_resid_t;
  s2.workspace = base + ws1;
  s2.workspace_bytes = ws2;
  rc = validate_stage(&s1);
  if (rc == PSD_OK) rc = validate_stage(&s2);
  if (rc != PSD_OK) return rc;
  const int policy = a->schedule != PSD_TWO_STAGE_DEFAULT ? a->schedule : t_two_stage_policy;
  bool separate = policy == PSD_TWO_STAGE_SEPARATE;
  int32_t* fill_out = nullptr;
  if (policy == PSD_TWO_STAGE_AUTO) {
    std::lock_guard<std::mutex> lock(ds->mu);
    if (ds->fill_host == nullptr) {
      void* h = nullptr;
      void* d = nullptr;
      if (cudaHostAlloc(&h, kFillCap * sizeof(int32_t), cudaHostAllocMapped) == cudaSuccess &&
          cudaHostGetDevicePointer(&d, h, 0) == cudaSuccess) {
        ds->fill_host = static_cast<int32_t*>(h);
        ds->fill_dev = static_cast<int32_t*>(d);
      } else {
        cudaGetLastError();   // no mapped memory: stay with two launches
      }
    }
    if (ds->fill_host != nullptr) {
      const int n = B < kFillCap ? B : kFillCap;
      const long long rows = static_cast<long long>(B) * (K_d + K_q);
      if (ds->fill_B == B && ds->fill_Kq == K_q && rows >= 1024) {
        long long filled = 0;
        const volatile int32_t* f = ds->fill_host;
        for (int i = 0; i < n; ++i) { const int v = f[i]; filled += v < 0 ? 0 : (v > K_q ? K_q : v); }
        // rows the stage-by-stage schedule would skip, as a share of all rows
        const double skipped = (1.0 - static_cast<double>(filled) / (static_cast<double>(n) * K_q)) * K_q / (K_d + K_q);
        separate = skipped > 0.10;
      } else {
        for (int i = 0; i < n; ++i) ds->fill_host[i] = K_q;   // unknown: assume full windows until stage 1 says otherwise
        ds->fill_B = B;
        ds->fill_Kq = K_q;
        ds->fill_calls = 0;
      }
      // The stores into mapped host memory cost the finalisation a few microseconds: the lengths are asked for on
      // every sixteenth call while windows are full, on every fourth while the call runs stage by stage (which is
      // how long a change of regime can go unnoticed).
      if ((ds->fill_calls++ % (separate ? 4u : 16u)) == 0u) fill_out = ds->fill_dev;
    }
  }
  const int variant = a->kernel_variant;
  const bool resid_any = a->out_resid_q != nullptr || a->out_resid_t != nullptr;
  int onepass = 0;
  if (separate) {
    // stage by stage: stage 2's statistics run after stage 1 has fixed the windows and skip the rows beyond them.
    // Both launches take the cluster size the single-launch schedule would pick, so a row's vocabulary is
    // cut into the same slices and its statistics come out bit-identical under either policy.
    {
      StageParams PS = make_params(&s1, s1.workspace, nullptr);
      const StageParams Q = make_params(&s2, s2.workspace, nullptr);
      PS.small2 = Q.small; PS.large2 = Q.large;
      PS.seq_stride_small2 = Q.seq_stride_small; PS.seq_stride_large2 = Q.seq_stride_large;
      PS.K2 = K_q;
      psd::ClusterGeom g{};
      if (variant != PSD_KERNEL_BASELINE && psd::cluster_geometry(PS, dtype, 0, false, false, &g)) s1.cluster_size = s2.cluster_size = g.cs;
      onepass = (variant == PSD_KERNEL_AUTO && psd::onepass_applies(PS, dtype, resid_any)) ? 1 : 0;
    }
    rc = run_stage_locked(&s1, ss, status, stream, window, n_window, K_q, fill_out, onepass);
    if (rc != PSD_OK) return rc;
    return run_stage_locked(&s2, ss, status, stream, nullptr, nullptr, 0, nullptr, onepass);
  }
  // Two launches for the whole pyramid. The statistics of both stages are independent of the stage-1
  // outcome (only the token looked up in a row and the window length depend on it), so one launch of
  // the statistics kernel covers the B*K_d stage-1 rows and the B*K_q stage-2 rows; one finalisation
  // kernel then runs stage 1, builds the window, and runs stage 2 per sequence.
  StageParams P1 = make_params(&s1, s1.workspace, status);
  P1.window = window;
  P1.n_window = n_window;
  P1.K_window = K_q;
  P1.fill_out = fill_out;
  P1.fill_cap = kFillCap;
  const StageParams P2 = make_params(&s2, s2.workspace, status);
  StageParams PS = P1;
  PS.small2 = P2.small;
  PS.large2 = P2.large;
  PS.seq_stride_small2 = P2.seq_stride_small;
  PS.seq_stride_large2 = P2.seq_stride_large;
  PS.K2 = K_q;
  PS.stats2 = P2.stats;
  rc = launch_rowstats(PS, dtype, variant, 0, stream, policy == PSD_TWO_STAGE_FUSED_ROWS || policy == PSD_TWO_STAGE_AUTO,
                       P1.out_resid_mass != nullptr || P2.out_resid_mass != nullptr);
  if (rc != PSD_OK) return rc;
  if (a->mode_t == PSD_FUZZY && split_finalize(2ll * B, V, P1.bonus != 0 || P2.bonus != 0, ss))
    return launch_finalize_split(P1, P2, 2, dtype, stream, ss);
  {
    TimedLaunch timed(stream, 1);
    cudaError_t e;
    if (a->mode_t == PSD_FUZZY) {
      // threshold rule in stage 2: it needs nothing of stage 1's drawn token, the stages run side by side
      const int cl = fin_cluster_size(2ll * B);
      if (dtype == PSD_F32) e = PSD_FIN_DISPATCH(finalize_pyramid_split_kernel, float, cl, 2u * B, stream, P1, P2);
      else e = PSD_FIN_DISPATCH(finalize_pyramid_split_kernel, __nv_bfloat16, cl, 2u * B, stream, P1, P2);
    } else {
      const int cl = fin_cluster_size(B);
      if (dtype == PSD_F32) e = PSD_FIN_DISPATCH(finalize_pyramid_kernel, float, cl, static_cast<unsigned>(B), stream, P1, P2);
      else e = PSD_FIN_DISPATCH(finalize_pyramid_kernel, __nv_bfloat16, cl, static_cast<unsigned>(B), stream, P1, P2);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e != cudaSuccess) { cudaGetLastError(); return PSD_ERR_CUDA; }
  }
  return check_launch();
}

cudaStream_t pick_stream(const psd_pyramid_args* a) {
  if (a->stream != nullptr || a->use_stream_field) return static_cast<cudaStream_t>(a->stream);
  return t_stream;
}

int verify_two_stage(const psd_pyramid_args* a) {
  int rc = validate_pyramid(a);
  if (rc != PSD_OK) return rc;
  if (a->B == 0) return PSD_OK;
  const cudaStream_t stream = pick_stream(a);
  if (a->workspace != nullptr) {
    int* status = reinterpret_cast<int*>(static_cast<char*>(a->workspace) + pyramid_workspace_bytes(a->B, a->K_d, a->K_q) - kAlign);
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return PSD_ERR_CUDA;
    t_last_scratch = nullptr; t_last_status = status; t_last_stream = stream;
    return verify_two_stage_locked(a, nullptr, status, stream);
  }
  StreamScratch* ss = nullptr;
  rc = scratch_for(stream, &ss);
  if (rc != PSD_OK) return rc;
  std::lock_guard<std::mutex> lock(ss->mu);
  rc = ensure_status(ss);
  if (rc != PSD_OK) return rc;
  t_last_scratch = ss; t_last_status = ss->status; t_last_stream = stream;
  return verify_two_stage_locked(a, ss, ss->status, stream);
}

psd_pyramid_args basic_pyramid_args(const void* logits_draft, const void* logits_qual, const void* logits_target,
                                    const int32_t* draft_tokens, int B, int K_d, int K_q, int V, int dtype, float tau_q,
                                    float tau_t, int mode, uint64_t seed, uint64_t offset, int32_t* out_accept_len_q,
                                    int32_t* out_next_token_q, int32_t* out_accept_len, int32_t* out_next_token) {
  psd_pyramid_args a;
  std::memset(&a, 0, sizeof(a));
  a.struct_size = sizeof(a);
  a.dtype = dtype;
  a.logits_draft = logits_draft; a.logits_qual = logits_qual; a.logits_target = logits_target;
  a.draft_tokens = draft_tokens;
  a.B = B; a.K_d = K_d; a.K_q = K_q; a.V = V;
  a.mode_q = a.mode_t = mode;
  a.tau_q = tau_q; a.tau_t = tau_t;
  a.div_kind = PSD_DIV_JS;
  a.philox_seed = seed; a.philox_offset = offset;
  a.out_accept_len_q = out_accept_len_q; a.out_next_token_q = out_next_token_q;
  a.out_accept_len = out_accept_len; a.out_next_token = out_next_token;
  return a;
}

}  // namespace

extern "C" {

int pyramidsd_verify_stage_ex(const psd_stage_args* args) { return run_stage(args); }

int pyramidsd_verify_stage(const void* logits_small, const void* logits_large, const int32_t* draft_tokens,
                           int B, int K, int V, psd_dtype dtype, float threshold, psd_mode mode,
                           uint64_t philox_seed, uint64_t offset, int32_t* out_accept_len,
                           int32_t* out_next_token) {
  psd_stage_args a;
  std::memset(&a, 0, sizeof(a));
  a.struct_size = sizeof(a);
  a.dtype = dtype;
  a.logits_small = logits_small;
  a.logits_large = logits_large;
  a.tokens = draft_tokens;
  a.B = B; a.K = K; a.V = V;
  a.mode = mode;
  a.div_kind = PSD_DIV_JS;
  a.threshold = threshold;
  a.philox_seed = philox_seed;
  a.philox_offset = offset;
  a.out_accept_len = out_accept_len;
  a.out_next_token = out_next_token;
  return run_stage(&a);
}

int pyramidsd_verify_ex(const psd_pyramid_args* args) { return verify_two_stage(args); }

int pyramidsd_verify(const void* logits_draft, const void* logits_qual, const void* logits_target,
                     const int32_t* draft_tokens, int B, int K_d, int K_q, int V, psd_dtype dtype,
                     float tau_q, float tau_t, psd_mode mode, uint64_t philox_seed, uint64_t offset,
                     int32_t* out_accept_len_q, int32_t* out_next_token_q, int32_t* out_accept_len,
                     int32_t* out_next_token) {
  const psd_pyramid_args a = basic_pyramid_args(logits_draft, logits_qual, logits_target, draft_tokens, B, K_d, K_q, V, dtype,
                                                tau_q, tau_t, mode, philox_seed, offset, out_accept_len_q, out_next_token_q,
                                                out_accept_len, out_next_token);
  return verify_two_stage(&a);
}

int pyramidsd_verify_bonus(const void* logits_draft, const void* logits_qual, const void* logits_target,
                           const int32_t* draft_tokens, int B, int K_d, int K_q, int V, psd_dtype dtype,
                           float tau_q, float tau_t, psd_mode mode, uint64_t philox_seed, uint64_t offset,
                           int32_t* out_accept_len_q, int32_t* out_next_token_q, int32_t* out_accept_len,
                           int32_t* out_next_token) {
  psd_pyramid_args a = basic_pyramid_args(logits_draft, logits_qual, logits_target, draft_tokens, B, K_d, K_q, V, dtype,
                                          tau_q, tau_t, mode, philox_seed, offset, out_accept_len_q, out_next_token_q,
                                          out_accept_len, out_next_token);
  a.target_has_bonus_row = 1;
  return verify_two_stage(&a);
}

int pyramidsd_verify_host(const void* logits_draft, const void* logits_qual, const void* logits_target,
                          const int32_t* draft_tokens, int B, int K_d, int K_q, int V, psd_dtype dtype,
                          float tau_q, float tau_t, psd_mode mode, uint64_t philox_seed, uint64_t offset,
                          int32_t* out_accept_len_q, int32_t* out_next_token_q, int32_t* out_accept_len,
                          int32_t* out_next_token) {
  psd_pyramid_args a = basic_pyramid_args(logits_draft, logits_qual, logits_target, draft_tokens, B, K_d, K_q, V, dtype,
                                          tau_q, tau_t, mode, philox_seed, offset, out_accept_len_q, out_next_token_q,
                                          out_accept_len, out_next_token);
  int rc = validate_pyramid(&a);
  if (rc != PSD_OK) return rc;
  if (B == 0) return PSD_OK;
  const cudaStream_t s = t_stream;
  StreamScratch* ss = nullptr;
  rc = scratch_for(s, &ss);
  if (rc != PSD_OK) return rc;
  std::lock_guard<std::mutex> lock(ss->mu);
  rc = ensure_status(ss);
  if (rc != PSD_OK) return rc;
  t_last_scratch = ss; t_last_status = ss->status; t_last_stream = s;
  const size_t es = elem_size(dtype);
  const size_t n_d = static_cast<size_t>(B) * K_d * V * es, n_t = static_cast<size_t>(B) * K_q * V * es;
  const size_t n_tok = static_cast<size_t>(B) * K_d * 4;
  const size_t want[4] = {n_d, n_d, n_t, n_tok};
  for (int i = 0; i < 4; ++i) {
    rc = grow(ss, &ss->stage[i], &ss->stage_bytes[i], want[i]);
    if (rc != PSD_OK) return rc;
  }
  rc = grow(ss, &ss->out4, &ss->out4_bytes, static_cast<size_t>(4) * B * 4);
  if (rc != PSD_OK) return rc;
  const void* src[4] = {logits_draft, logits_qual, logits_target, draft_tokens};
  for (int i = 0; i < 4; ++i)
    if (cudaMemcpyAsync(ss->stage[i], src[i], want[i], cudaMemcpyHostToDevice, s) != cudaSuccess) return PSD_ERR_CUDA;
  int32_t* o = static_cast<int32_t*>(ss->out4);
  a.logits_draft = ss->stage[0]; a.logits_qual = ss->stage[1]; a.logits_target = ss->stage[2];
  a.draft_tokens = static_cast<const int32_t*>(ss->stage[3]);
  a.out_accept_len_q = o; a.out_next_token_q = o + B; a.out_accept_len = o + 2 * B; a.out_next_token = o + 3 * B;
  rc = verify_two_stage_locked(&a, ss, ss->status, s);
  if (rc != PSD_OK) return rc;
  int32_t* dst[4] = {out_accept_len_q, out_next_token_q, out_accept_len, out_next_token};
  for (int i = 0; i < 4; ++i)
    if (cudaMemcpyAsync(dst[i], o + static_cast<size_t>(i) * B, static_cast<size_t>(B) * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)
      return PSD_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
}

int pyramidsd_verify_stage_noalloc(const void* logits_small, const void* logits_large, const int32_t* draft_tokens,
                                   int B, int K, int V, psd_dtype dtype, float threshold, psd_mode mode,
                                   uint64_t philox_seed, uint64_t offset, int32_t* out_accept_len,
                                   int32_t* out_next_token, int32_t* out_wait_timeout, void* cuda_stream) {
  if (B < 0 || K < 0) return PSD_ERR_INVALID_ARG;
  if (static_cast<long long>(B) * K > PSD_NOALLOC_MAX_ROWS) {
    std::fprintf(stderr, "pyramidsd_verify_stage_noalloc: B * K = %lld rows exceed the built-in scratch of %d rows\n",
                 static_cast<long long>(B) * K, PSD_NOALLOC_MAX_ROWS);
    return PSD_ERR_UNSUPPORTED;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSD_ERR_CUDA;
  void* scratch = nullptr;
  {
    // first call on this device: look the array's device address up, with this device current
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (g_noalloc_ptr[dev] == nullptr) {
      void* p = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
      if (e != cudaSuccess || p == nullptr) {
        std::fprintf(stderr, "pyramidsd_verify_stage_noalloc: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
        cudaGetLastError();
        return PSD_ERR_CUDA;
      }
      g_noalloc_ptr[dev] = p;
    }
    scratch = g_noalloc_ptr[dev];
  }
  psd_stage_args a;
  std::memset(&a, 0, sizeof(a));
  a.struct_size = sizeof(a);
  a.dtype = dtype;
  a.logits_small = logits_small;
  a.logits_large = logits_large;
  a.tokens = draft_tokens;
  a.B = B; a.K = K; a.V = V;
  a.mode = mode;
  a.div_kind = PSD_DIV_JS;
  a.threshold = threshold;
  a.philox_seed = philox_seed;
  a.philox_offset = offset;
  a.out_accept_len = out_accept_len;
  a.out_next_token = out_next_token;
  int rc = validate_stage(&a);
  if (rc != PSD_OK) return rc;
  if (B == 0) return PSD_OK;
  const cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int* flag = reinterpret_cast<int*>(static_cast<unsigned char*>(scratch) + kNoAllocStatsBytes);
  // the flag is the one thing that has to start at zero; the statistics of every row read are written first
  if (cudaMemsetAsync(flag, 0, sizeof(int), stream) != cudaSuccess) return PSD_ERR_CUDA;
  const StageParams P = make_params(&a, scratch, flag);
  if (K > 0) {
    rc = launch_rowstats(P, dtype, PSD_KERNEL_AUTO, 0, stream);
    if (rc != PSD_OK) return rc;
  }
  rc = launch_finalize(P, dtype, stream);
  if (rc != PSD_OK) return rc;
  if (out_wait_timeout != nullptr &&
      cudaMemcpyAsync(out_wait_timeout, flag, sizeof(int), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
    return PSD_ERR_CUDA;
  return PSD_OK;
}

int pyramidsd_verify_fused_lmhead_ex(const psd_lmhead_args* args) {
  if (args == nullptr || args->struct_size != sizeof(psd_lmhead_args)) return PSD_ERR_INVALID_ARG;
  if (args->tile_variant < PSD_LMHEAD_TILES_AUTO || args->tile_variant > PSD_LMHEAD_TILES_ONE_SM || args->seq_index_base < 0) return PSD_ERR_INVALID_ARG;
  if (!valid_div(args->div_kind) || args->reserved0 != 0) return PSD_ERR_INVALID_ARG;
  if (args->div_kind == PSD_DIV_TV) return PSD_ERR_UNSUPPORTED;
  const bool kl = args->div_kind == PSD_DIV_KL;
  const void* hidden = args->hidden;
  const void* w_t = args->w_t;
  const void* logits_small = args->logits_small;
  const int32_t* tokens = args->tokens;
  const int B = args->B, K = args->K, d_model = args->d_model, V = args->V, mode = args->mode;
  const float threshold = args->threshold;
  const uint64_t philox_seed = args->philox_seed, offset = args->philox_offset;
  int32_t* out_accept_len = args->out_accept_len;
  int32_t* out_next_token = args->out_next_token;
  float* out_div = args->out_div;
  float* out_resid_mass = args->out_resid_mass;
  void* cuda_stream = args->stream;
  if (!valid_mode(mode) || B < 0 || K < 0 || K > 32 || V < 1 || d_model < 1 || std::isnan(threshold)) return PSD_ERR_INVALID_ARG;
  const long long M = static_cast<long long>(B) * K;
  if ((d_model % psd::kLmK) != 0) return PSD_ERR_UNSUPPORTED;
  if (B == 0) return PSD_OK;
  if (!out_accept_len || !out_next_token) return PSD_ERR_INVALID_ARG;
  if (K > 0 && (!hidden || !w_t || !logits_small || !tokens)) return PSD_ERR_INVALID_ARG;
  if (((reinterpret_cast<uintptr_t>(hidden) | reinterpret_cast<uintptr_t>(w_t)) & 15u) != 0) return PSD_ERR_UNSUPPORTED;
  const cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (K == 0) {
    // nothing to verify: every sequence accepts its empty window
    if (cudaMemsetAsync(out_accept_len, 0, static_cast<size_t>(B) * 4, stream) != cudaSuccess) return PSD_ERR_CUDA;
    if (cudaMemsetAsync(out_next_token, 0xff, static_cast<size_t>(B) * 4, stream) != cudaSuccess) return PSD_ERR_CUDA;
    return PSD_OK;
  }
  StreamScratch* ss = nullptr;
  int rc = scratch_for(stream, &ss);
  if (rc != PSD_OK) return rc;
  std::lock_guard<std::mutex> lock(ss->mu);
  const int n_tiles = (V + psd::kLmN - 1) / psd::kLmN;
  const size_t per = static_cast<size_t>(M) * n_tiles;
  const size_t bytes = align_up(per * sizeof(float2)) * 2 + align_up(per * sizeof(float4)) + align_up(static_cast<size_t>(M) * sizeof(float4)) +
                       align_up(per * sizeof(float)) + align_up(static_cast<size_t>(M) * sizeof(float)) + kAlign;
  rc = ensure_status(ss);
  if (rc != PSD_OK) return rc;
  t_last_scratch = ss; t_last_status = ss->status; t_last_stream = stream;
  rc = grow(ss, &ss->lm_ws, &ss->lm_ws_bytes, bytes);
  if (rc != PSD_OK) return rc;
  // tensor maps: hidden [M, d] and W^T [V, d], bf16, K innermost, boxes of 64 x 256 / 64 x 128, 128-byte swizzle
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) fn = nullptr;
    return reinterpret_cast<EncodeFn>(fn);
  }();
  if (encode == nullptr) return PSD_ERR_CUDA;
  CUtensorMap map_a, map_b;
  {
    const cuuint64_t dims_a[2] = {static_cast<cuuint64_t>(d_model), static_cast<cuuint64_t>(M)};
    const cuuint64_t dims_b[2] = {static_cast<cuuint64_t>(d_model), static_cast<cuuint64_t>(V)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d_model) * 2};
    const cuuint32_t box_a[2] = {psd::kLmK, psd::kLmM}, box_b[2] = {psd::kLmK, psd::kLmN}, estr[2] = {1, 1};
    if (encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims_a, strides, box_a, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return PSD_ERR_CUDA;
    if (encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w_t), dims_b, strides, box_b, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return PSD_ERR_CUDA;
  }
  char* ws = static_cast<char*>(ss->lm_ws);
  psd::LmParams L{};
  L.small = static_cast<const __nv_bfloat16*>(logits_small);
  L.tokens = tokens;
  L.M = static_cast<int>(M); L.d = d_model; L.V = V; L.n_tiles = n_tiles;
  L.c = 1.4426950408889634f;
  L.part_large = reinterpret_cast<float2*>(ws); ws += align_up(per * sizeof(float2));
  L.part_small = reinterpret_cast<float2*>(ws); ws += align_up(per * sizeof(float2));
  L.part_div = reinterpret_cast<float4*>(ws); ws += align_up(per * sizeof(float4));
  L.row_lse = reinterpret_cast<float4*>(ws); ws += align_up(static_cast<size_t>(M) * sizeof(float4));
  L.status = ss->status;
  if (kl) {
    L.part_t = reinterpret_cast<float*>(ws); ws += align_up(per * sizeof(float));
    L.row_div = reinterpret_cast<float*>(ws); ws += align_up(static_cast<size_t>(M) * sizeof(float));
    L.need_sweep2 = reinterpret_cast<int*>(ws);
    // the residual masses are wanted as an output: the second sweep runs whatever the accept scan finds
    if (cudaMemsetAsync(L.need_sweep2, out_resid_mass != nullptr ? 1 : 0, sizeof(int), stream) != cudaSuccess) return PSD_ERR_CUDA;
  }
  static bool attr_set[kMaxDevices] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev]) {
    const int one = static_cast<int>(psd::kLmSmemBytes), two = static_cast<int>(psd::kLm2SmemBytes);
    const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
    if (cudaFuncSetAttribute(psd::lmhead_sweep_kernel<1, false>, at, one) != cudaSuccess ||
        cudaFuncSetAttribute(psd::lmhead_sweep_kernel<1, true>, at, one) != cudaSuccess ||
        cudaFuncSetAttribute(psd::lmhead_sweep_kernel<2, false>, at, one) != cudaSuccess ||
        cudaFuncSetAttribute(psd::lmhead_sweep2sm_kernel<1, false>, at, two) != cudaSuccess ||
        cudaFuncSetAttribute(psd::lmhead_sweep2sm_kernel<1, true>, at, two) != cudaSuccess ||
        cudaFuncSetAttribute(psd::lmhead_sweep2sm_kernel<2, false>, at, two) != cudaSuccess) {
      cudaGetLastError();
      return PSD_ERR_CUDA;
    }
    attr_set[dev] = true;
  }
  int sms = psd::cluster_sm_count();
  if (sms <= 0) sms = 1;
  // the two-SM (cta_group::2) sweeps are the default
  const bool use_pair = args->tile_variant != PSD_LMHEAD_TILES_ONE_SM;
  CUtensorMap map_a2, map_b2;   // the pair's A / B boxes are 64 x 128
  if (use_pair) {
    const cuuint64_t dims_a[2] = {static_cast<cuuint64_t>(d_model), static_cast<cuuint64_t>(M)};
    const cuuint64_t dims_b[2] = {static_cast<cuuint64_t>(d_model), static_cast<cuuint64_t>(V)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d_model) * 2};
    const cuuint32_t box[2] = {psd::kLmK, 128}, estr[2] = {1, 1};
    if (encode(&map_a2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims_a, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return PSD_ERR_CUDA;
    if (encode(&map_b2, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w_t), dims_b, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return PSD_ERR_CUDA;
  }
  const int n_tiles2 = (n_tiles + 1) / 2;
  const int pairs = n_tiles2 < sms / 2 ? n_tiles2 : sms / 2;
  const unsigned grid_one = static_cast<unsigned>(n_tiles < sms ? n_tiles : sms);
  // one GEMM sweep over every block of 256 rows (the weight is streamed once per block and sweep)
  auto launch_sweep = [&](int sweep) -> bool {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    if (use_pair) {
      cfg.gridDim = dim3(static_cast<unsigned>(2 * (pairs > 0 ? pairs : 1)));
      cfg.dynamicSmemBytes = psd::kLm2SmemBytes;
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      cfg.attrs = at;
      cfg.numAttrs = 1;
    } else {
      cfg.gridDim = dim3(grid_one);
      cfg.dynamicSmemBytes = psd::kLmSmemBytes;
    }
    cfg.blockDim = dim3(psd::kLmThreads);
    cfg.stream = stream;
    for (int r0 = 0; r0 < M; r0 += psd::kLmM) {
      L.row0 = r0;
      cudaError_t e;
      if (use_pair) {
        if (sweep == 2) e = cudaLaunchKernelEx(&cfg, psd::lmhead_sweep2sm_kernel<2, false>, map_a2, map_b2, L);
        else if (kl) e = cudaLaunchKernelEx(&cfg, psd::lmhead_sweep2sm_kernel<1, true>, map_a2, map_b2, L);
        else e = cudaLaunchKernelEx(&cfg, psd::lmhead_sweep2sm_kernel<1, false>, map_a2, map_b2, L);
      } else {
        if (sweep == 2) e = cudaLaunchKernelEx(&cfg, psd::lmhead_sweep_kernel<2, false>, map_a, map_b, L);
        else if (kl) e = cudaLaunchKernelEx(&cfg, psd::lmhead_sweep_kernel<1, true>, map_a, map_b, L);
        else e = cudaLaunchKernelEx(&cfg, psd::lmhead_sweep_kernel<1, false>, map_a, map_b, L);
      }
      if (e != cudaSuccess) { cudaGetLastError(); return false; }
    }
    L.row0 = 0;
    return true;
  };
  psd::LmFinalParams F{};
  F.hidden = static_cast<const __nv_bfloat16*>(hidden);
  F.w_t = static_cast<const __nv_bfloat16*>(w_t);
  F.B = B; F.K = K;
  F.threshold = threshold;
  F.mode = mode;
  F.seed = philox_seed; F.offset = offset;
  F.seq_base = args->seq_index_base;
  F.out_accept_len = out_accept_len;
  F.out_next_token = out_next_token;
  F.out_div = out_div;
  F.out_resid = out_resid_mass;
  uint64_t launches = 0;
  {
    TimedLaunch timed(stream, 0);
    if (!launch_sweep(1)) return PSD_ERR_CUDA;
    psd::lmhead_reduce_kernel<<<static_cast<unsigned>((M + 7) / 8), 256, 0, stream>>>(L);
    if (kl) {
      // Kullback-Leibler: the divergences are known after one sweep. The accept scan says whether any rejected row
      // needs residual masses; only then does the second sweep do anything.
      F.lm = L;
      F.kl_phase = 1;
      psd::lmhead_final_kernel<<<static_cast<unsigned>(B), 256, 0, stream>>>(F);
      ++launches;
    }
    if (!launch_sweep(2)) return PSD_ERR_CUDA;
  }
  F.lm = L;
  F.kl_phase = kl ? 2 : 0;
  {
    TimedLaunch timed(stream, 1);
    psd::lmhead_final_kernel<<<static_cast<unsigned>(B), 256, 0, stream>>>(F);
  }
  g_launches.fetch_add(launches + 2 + 2 * static_cast<uint64_t>((M + psd::kLmM - 1) / psd::kLmM), std::memory_order_relaxed);
  return check_launch();
}

int pyramidsd_verify_fused_lmhead(const void* hidden, const void* w_t, const void* logits_small,
                                  const int32_t* tokens, int B, int K, int d_model, int V, float threshold,
                                  psd_mode mode, uint64_t philox_seed, uint64_t offset, int32_t* out_accept_len,
                                  int32_t* out_next_token, float* out_div, float* out_resid_mass, void* cuda_stream) {
  psd_lmhead_args a;
  std::memset(&a, 0, sizeof(a));
  a.struct_size = sizeof(a);
  a.hidden = hidden; a.w_t = w_t; a.logits_small = logits_small; a.tokens = tokens;
  a.B = B; a.K = K; a.d_model = d_model; a.V = V;
  a.threshold = threshold;
  a.mode = mode;
  a.philox_seed = philox_seed; a.philox_offset = offset;
  a.out_accept_len = out_accept_len; a.out_next_token = out_next_token;
  a.out_div = out_div; a.out_resid_mass = out_resid_mass;
  a.stream = cuda_stream;
  return pyramidsd_verify_fused_lmhead_ex(&a);
}

double pyramidsd_model_sd_throughput(double beta, double ell, double v_small, double v_large) {
  if (!(beta >= 0.0 && beta <= 1.0) || !(ell > 0.0) || !(v_small > 0.0) || !(v_large > 0.0)) return std::nan("");
  return beta * (ell + 1.0) / (ell / v_small + 1.0 / v_large);
}

double pyramidsd_model_psd_throughput(double beta_qd, double ell_d, double v_draft, double v_qual, double beta_tq,
                                      double ell_q, double v_target) {
  const double v_fsd = pyramidsd_model_sd_throughput(beta_qd, ell_d, v_draft, v_qual);
  if (!(v_fsd > 0.0)) return std::nan("");
  return pyramidsd_model_sd_throughput(beta_tq, ell_q, v_fsd, v_target);
}

int pyramidsd_row_uniforms(uint64_t philox_seed, uint64_t offset, int n_rows, float* out_u, float* out_u2) {
  if (n_rows < 0) return PSD_ERR_INVALID_ARG;
  if (n_rows == 0 || (!out_u && !out_u2)) return PSD_OK;
  row_uniforms_kernel<<<(n_rows + 255) / 256, 256, 0, t_stream>>>(philox_seed, offset, n_rows, out_u, out_u2);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return check_launch();
}

size_t pyramidsd_workspace_bytes(int B, int K, int V, psd_dtype dtype) {
  if (B < 0 || K < 0 || K > 32 || V < 1 || !valid_dtype(dtype)) return 0;
  return stage_workspace_bytes(B, K);
}

size_t pyramidsd_pyramid_workspace_bytes(int B, int K_d, int K_q, int V, psd_dtype dtype) {
  if (B < 0 || K_q < 1 || K_d < K_q || K_d > 32 || V < 1 || !valid_dtype(dtype)) return 0;
  return pyramid_workspace_bytes(B, K_d, K_q);
}

int pyramidsd_set_two_stage_policy(int policy) {
  if (policy < PSD_TWO_STAGE_DEFAULT || policy > PSD_TWO_STAGE_FUSED_ROWS) return PSD_ERR_INVALID_ARG;
  t_two_stage_policy = policy == PSD_TWO_STAGE_DEFAULT ? PSD_TWO_STAGE_AUTO : policy;
  return PSD_OK;
}

int pyramidsd_set_stream(void* cuda_stream) {
  t_stream = static_cast<cudaStream_t>(cuda_stream);
  return PSD_OK;
}

int pyramidsd_release_stream(void* cuda_stream) {
  const cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  DeviceState* ds = nullptr;
  int rc = current_device_state(&ds);
  if (rc != PSD_OK) return rc;
  std::lock_guard<std::mutex> table(ds->mu);
  for (auto& e : ds->streams) {
    if (!e.used || e.stream != stream) continue;
    std::lock_guard<std::mutex> lock(e.mu);
    if (cudaStreamSynchronize(stream) != cudaSuccess) return PSD_ERR_CUDA;
    void** owned[] = {&e.ws, reinterpret_cast<void**>(&e.status), &e.stage[0], &e.stage[1], &e.stage[2], &e.stage[3], &e.out4, &e.lm_ws, &e.draw};
    for (void** p : owned) {
      if (*p) cudaFree(*p);
      *p = nullptr;
    }
    e.ws_bytes = e.out4_bytes = e.lm_ws_bytes = e.draw_bytes = 0;
    for (size_t& b : e.stage_bytes) b = 0;
    if (t_last_scratch == &e) { t_last_scratch = nullptr; t_last_status = nullptr; }
    e.used = false;
    e.stream = nullptr;
  }
  return PSD_OK;
}

int pyramidsd_last_status(void) {
  if (t_last_status == nullptr) return cudaStreamSynchronize(t_stream) == cudaSuccess ? PSD_OK : PSD_ERR_CUDA;
  StreamScratch* ss = t_last_scratch;
  std::unique_lock<std::mutex> lock;
  if (ss != nullptr) lock = std::unique_lock<std::mutex>(ss->mu);
  if (cudaStreamSynchronize(t_last_stream) != cudaSuccess) return PSD_ERR_CUDA;
  int host = 0;
  if (cudaMemcpy(&host, t_last_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PSD_ERR_CUDA;
  if (host != 0) {
    cudaMemset(t_last_status, 0, sizeof(int));
    return PSD_ERR_TIMEOUT;
  }
  return PSD_OK;
}

int pyramidsd_selftest_wait_timeout(void* cuda_stream) {
  const cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  StreamScratch* ss = nullptr;
  int rc = scratch_for(stream, &ss);
  if (rc != PSD_OK) return rc;
  std::lock_guard<std::mutex> lock(ss->mu);
  rc = ensure_status(ss);
  if (rc != PSD_OK) return rc;
  t_last_scratch = ss; t_last_status = ss->status; t_last_stream = stream;
  psd::wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(ss->status);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return check_launch();
}

int pyramidsd_kernel_timing_begin(void) {
  t_timing.n = 0;
  t_timing.on = true;
  return PSD_OK;
}

int pyramidsd_kernel_timing_end(double* ms_rowstats, int* n_rowstats, double* ms_finalize, int* n_finalize) {
  Timing& t = t_timing;
  t.on = false;
  double ms[2] = {0.0, 0.0};
  int cnt[2] = {0, 0};
  for (int i = 0; i < t.n; ++i) {
    if (cudaEventSynchronize(t.ev[i][1]) != cudaSuccess) return PSD_ERR_CUDA;
    float f = 0.f;
    if (cudaEventElapsedTime(&f, t.ev[i][0], t.ev[i][1]) != cudaSuccess) return PSD_ERR_CUDA;
    ms[t.tag[i]] += f;
    cnt[t.tag[i]] += 1;
  }
  t.n = 0;
  if (ms_rowstats) *ms_rowstats = ms[0];
  if (n_rowstats) *n_rowstats = cnt[0];
  if (ms_finalize) *ms_finalize = ms[1];
  if (n_finalize) *n_finalize = cnt[1];
  return PSD_OK;
}

uint64_t pyramidsd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int pyramidsd_cluster_occupancy(int B, int K, int V, psd_dtype dtype, int* out_cluster_size, int* out_max_active_clusters) {
  if (B < 0 || K < 0 || K > 32 || V < 1 || !valid_dtype(dtype)) return PSD_ERR_INVALID_ARG;
  StageParams P{};
  P.B = B; P.K = K; P.V = V;
  P.seq_stride_small = P.seq_stride_large = static_cast<long long>(K) * V;
  P.div_kind = PSD_DIV_JS;
  psd::ClusterGeom g{};
  const bool ok = B > 0 && K > 0 && psd::cluster_geometry(P, dtype, 0, false, false, &g);
  if (out_cluster_size) *out_cluster_size = ok ? g.cs : 0;
  if (out_max_active_clusters) {
    *out_max_active_clusters = ok ? psd::cluster_max_active_any(dtype, PSD_DIV_JS, g.cs) : 0;
  }
  return PSD_OK;
}

const char* pyramidsd_version(void) { return "pyramidsd-b200 0.1.0 (sm_100a)"; }

const char* pyramidsd_status_string(int status) {
  switch (status) {
    case PSD_OK: return "ok";
    case PSD_ERR_INVALID_ARG: return "invalid argument";
    case PSD_ERR_UNSUPPORTED: return "unsupported shape or option";
    case PSD_ERR_WORKSPACE: return "workspace too small or misaligned";
    case PSD_ERR_CUDA: return "CUDA runtime error";
    case PSD_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

}  // extern "C"

// C-ABI layer: context, scratch management, plan caching and the call sequences of the public
// entry points declared in include/qv2.h.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#if defined(__has_include)
#if __has_include(<nvtx3/nvToolsExt.h>)
#include <nvtx3/nvToolsExt.h>
#define QV2_HAVE_NVTX 1
#endif
#endif

#include "qv2_common.cuh"

using namespace qv2;

namespace {
constexpr int kCodeRing = 4;     // pinned staging areas for the per-call table of code pointers
constexpr uint64_t kDefaultChunkBytes = 48ull << 20;
}

struct qv2_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  int sm_count = 1;
  GridCaps caps;               // largest useful grid of each persistent kernel on this device
  int last_cuda = 0;
  uint64_t launches = 0;
  uint64_t syncs = 0;          // host-side stream synchronisations this context has performed
  uint32_t live_graphs = 0;    // captured passes that hold addresses of this context's scratch
  bool log = false;            // QV2_LOG=1: one line per call on stderr
  uint32_t schedule = QV2_SCHEDULE_PHASE_MAJOR;
  uint64_t chunk_bytes = kDefaultChunkBytes;
  uint32_t fold_mode = QV2_FOLD_AUTO;
  bool dependent_launch = true;   // kernels of a pass are launched as programmatic dependents of one another

  // cached plan: rebuilt only when the descriptor bytes or the schedule change
  HostPlan plan;
  std::vector<uint8_t> plan_key;
  bool plan_valid = false;

  // device scratch
  TensorRec* d_tensors = nullptr; size_t cap_tensors = 0;
  Tile* d_tiles = nullptr;        size_t cap_tiles = 0;
  Tile* d_hist_tiles = nullptr;   size_t cap_hist_tiles = 0;
  Tile* d_ghist_tiles = nullptr;  size_t cap_ghist_tiles = 0;   // per-group histogram mode
  uint32_t* d_ghist_owner = nullptr; size_t cap_ghist_owner = 0;
  unsigned long long* d_ghist = nullptr; size_t cap_ghist = 0;  // used when the caller passes no group_hist
  double2* d_partials = nullptr;  size_t cap_slots = 0;
  uint2* d_rslots = nullptr;      size_t cap_rslots = 0;
  double* d_partials_xe = nullptr; size_t cap_slots_xe = 0;   // sum x*e slots, cosine only
  unsigned long long* d_kl_hist = nullptr; size_t cap_kl_hist = 0;   // used when the caller passes no hists
  float* d_tensor_absmax = nullptr; size_t cap_absmax = 0;
  // accumulators that are zero between passes (cleared when a plan is made resident, and by the
  // CTA that consumes them afterwards)
  uint32_t* d_keys = nullptr;     size_t cap_keys = 0;         // kmin then kmax, total_groups each
  unsigned long long* d_nf_acc = nullptr; size_t cap_nf = 0;   // per tensor
  unsigned long long* d_hist_acc = nullptr; size_t cap_hist_acc = 0;   // 2048 per percentile tensor
  uint32_t* d_tickets = nullptr;  size_t cap_tickets = 0;      // 3 per tensor: range, histogram, metrics
  uint8_t** d_codes = nullptr;    size_t cap_codes = 0;        // per-tensor code buffers of the current call
  double* d_rank = nullptr;                                    // 2 * kMaxRankLayers doubles
  // pinned host staging for the plan upload
  uint8_t* h_pinned = nullptr;    size_t cap_pinned = 0;
  // pinned ring for the code-pointer table: a call fills the next area and copies it on the
  // stream; the area's event tells when it may be refilled
  uint8_t** h_codes[kCodeRing] = {}; size_t cap_h_codes = 0;
  cudaEvent_t code_ev[kCodeRing] = {};
  uint32_t code_next = 0;
  // qv2_set_phase_timing: events around the range and histogram phases of qv2_calibrate
  bool phase_timing = false;
  bool phase_marks_valid = false;
  cudaEvent_t phase_ev[3] = {};
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

// A named range around each entry point for timeline tools; compiled out without the NVTX headers.
struct TraceRange {
#ifdef QV2_HAVE_NVTX
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
#else
  explicit TraceRange(const char*) {}
#endif
};

// QV2_LOG=1: one line per call on stderr (host side only; nothing is read back from the device).
void log_call(const qv2_ctx* c, const char* call, uint32_t n_tensors, uint64_t launches_before, int status) {
  if (!c->log) return;
  std::fprintf(stderr, "qv2: %s tensors=%u tiles=%zu stages=%zu launches=%llu status=%d (%s)\n", call, n_tensors,
               c->plan_valid ? c->plan.tiles.size() : (size_t)0, c->plan_valid ? c->plan.stages.size() : (size_t)0,
               (unsigned long long)(c->launches - launches_before), status, qv2_status_string(status));
}

int cuda_fail(qv2_ctx* c, cudaError_t e) {
  c->last_cuda = (int)e;
  c->plan_valid = false;          // a pass that stopped half-way may leave accumulators dirty: start over
  return e == cudaErrorMemoryAllocation ? QV2_ERR_NOMEM : QV2_ERR_CUDA;
}

#define QV2_CUDA(c, expr)                              \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) return cuda_fail((c), e__);\
  } while (0)

// graph_held: a captured pass may hold the address of this buffer, so it must not move while one
// is alive.
template <class T>
int grow(qv2_ctx* c, T** p, size_t* cap, size_t need, bool graph_held = true) {
  if (need <= *cap) return QV2_OK;
  if (graph_held && c->live_graphs) return QV2_ERR_UNSUPPORTED;
  size_t want = need + need / 4 + 16;
  if (*p) { QV2_CUDA(c, cudaFree(*p)); *p = nullptr; *cap = 0; }
  QV2_CUDA(c, cudaMalloc((void**)p, want * sizeof(T)));
  *cap = want;
  return QV2_OK;
}

int grow_pinned(qv2_ctx* c, size_t need) {
  if (need <= c->cap_pinned) return QV2_OK;
  size_t want = need + need / 4 + 4096;
  if (c->h_pinned) { QV2_CUDA(c, cudaFreeHost(c->h_pinned)); c->h_pinned = nullptr; c->cap_pinned = 0; }
  QV2_CUDA(c, cudaMallocHost((void**)&c->h_pinned, want));
  c->cap_pinned = want;
  return QV2_OK;
}

int sync_stream(qv2_ctx* c) {
  ++c->syncs;
  QV2_CUDA(c, cudaStreamSynchronize(c->stream));
  return QV2_OK;
}

// Chunk size of the plan about to be built: 0 = phase-major (one stage).
//
// QV2_SCHEDULE_AUTO currently always answers phase-major.  Measured on a B200, a buffer that is read
// again is served from L2 at about 2.2 times the HBM rate only while it is at most ~32 MB (a
// persistent kernel re-reading 8..512 MB: 13-17 TB/s up to 32 MB, 9-13 TB/s at 48 MB, the HBM rate
// from 96 MB on), so the second and third pass over a stage can save at most half of their time
// on stages that small, while every stage adds launches of a few microseconds each and leaves the
// streaming kernels with one or two tiles per thread block.  On ResNet-18 shapes (batch 32) the
// chunked pass takes 0.38-0.56 ms against 0.27-0.30 ms phase-major, on ResNet-50 1.67-1.91 against
// 1.23 ms; it is kept for callers that ask for it.
uint64_t plan_chunk_bytes(const qv2_ctx* c, const qv2_tensor_desc*, uint32_t) {
  return c->schedule == QV2_SCHEDULE_L2_CHUNKED ? c->chunk_bytes : 0;
}

int ensure_plan_checked(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n);

// Makes ctx->plan describe descs and resident on the device.
int ensure_plan(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n) {
  try {
    return ensure_plan_checked(c, descs, n);
  } catch (const std::bad_alloc&) {          // host tables did not fit: nothing unwinds through the C ABI
    c->plan_valid = false;
    return QV2_ERR_NOMEM;
  }
}

int ensure_plan_checked(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n) {
  if (!descs) return QV2_ERR_NULL;
  if (n == 0 || n > 65535u) return QV2_ERR_SIZE;
  const size_t dbytes = (size_t)n * sizeof(qv2_tensor_desc);
  const uint64_t chunk = plan_chunk_bytes(c, descs, n);
  std::vector<uint8_t> key(dbytes + sizeof(chunk) + sizeof(c->fold_mode));
  std::memcpy(key.data(), descs, dbytes);
  std::memcpy(key.data() + dbytes, &chunk, sizeof(chunk));
  std::memcpy(key.data() + dbytes + sizeof(chunk), &c->fold_mode, sizeof(c->fold_mode));
  if (c->plan_valid && key == c->plan_key) return QV2_OK;
  // A captured pass replays with the tile tables and scratch addresses of the plan it was
  // captured with; another descriptor set would overwrite them under it.
  if (c->live_graphs) return QV2_ERR_UNSUPPORTED;

  HostPlan plan;
  int st = build_plan(descs, n, c->caps, chunk, c->fold_mode, &plan);
  if (st != QV2_OK) return st;
  // The previous upload may still be reading the pinned buffer, and buffers may be reallocated.
  if ((st = sync_stream(c)) != QV2_OK) return st;
  c->plan_valid = false;
  const size_t nt = plan.tensors.size(), ntl = plan.tiles.size(), nh = plan.hist_tiles.size();
  const size_t G = (size_t)plan.total_groups, nacc = (size_t)plan.n_hist * kBins;
  if ((st = grow(c, &c->d_tensors, &c->cap_tensors, nt)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_tiles, &c->cap_tiles, ntl ? ntl : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_hist_tiles, &c->cap_hist_tiles, nh ? nh : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_partials, &c->cap_slots, plan.total_slots ? plan.total_slots : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_rslots, &c->cap_rslots, plan.total_rslots ? plan.total_rslots : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_tensor_absmax, &c->cap_absmax, nt)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_keys, &c->cap_keys, 2 * G)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_nf_acc, &c->cap_nf, nt)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_hist_acc, &c->cap_hist_acc, nacc ? nacc : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_tickets, &c->cap_tickets, 3 * nt)) != QV2_OK) return st;
  const size_t ngt = plan.ghist_tiles.size(), ngo = plan.ghist_owner.size();
  if ((st = grow(c, &c->d_ghist_tiles, &c->cap_ghist_tiles, ngt ? ngt : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_ghist_owner, &c->cap_ghist_owner, ngo ? ngo : 1)) != QV2_OK) return st;
  const size_t b0 = nt * sizeof(TensorRec), b1 = ntl * sizeof(Tile), b2 = nh * sizeof(Tile);
  const size_t b3 = ngt * sizeof(Tile), b4 = ngo * sizeof(uint32_t);
  if ((st = grow_pinned(c, b0 + b1 + b2 + b3 + b4)) != QV2_OK) return st;
  std::memcpy(c->h_pinned, plan.tensors.data(), b0);
  if (b1) std::memcpy(c->h_pinned + b0, plan.tiles.data(), b1);
  if (b2) std::memcpy(c->h_pinned + b0 + b1, plan.hist_tiles.data(), b2);
  QV2_CUDA(c, cudaMemcpyAsync(c->d_tensors, c->h_pinned, b0, cudaMemcpyHostToDevice, c->stream));
  if (b1) QV2_CUDA(c, cudaMemcpyAsync(c->d_tiles, c->h_pinned + b0, b1, cudaMemcpyHostToDevice, c->stream));
  if (b2) QV2_CUDA(c, cudaMemcpyAsync(c->d_hist_tiles, c->h_pinned + b0 + b1, b2, cudaMemcpyHostToDevice, c->stream));
  if (b3) {
    std::memcpy(c->h_pinned + b0 + b1 + b2, plan.ghist_tiles.data(), b3);
    std::memcpy(c->h_pinned + b0 + b1 + b2 + b3, plan.ghist_owner.data(), b4);
    QV2_CUDA(c, cudaMemcpyAsync(c->d_ghist_tiles, c->h_pinned + b0 + b1 + b2, b3, cudaMemcpyHostToDevice, c->stream));
    QV2_CUDA(c, cudaMemcpyAsync(c->d_ghist_owner, c->h_pinned + b0 + b1 + b2 + b3, b4, cudaMemcpyHostToDevice, c->stream));
  }
  // every accumulator starts at zero; from here on the kernels keep them so
  QV2_CUDA(c, cudaMemsetAsync(c->d_keys, 0, 2 * G * sizeof(uint32_t), c->stream));
  QV2_CUDA(c, cudaMemsetAsync(c->d_nf_acc, 0, nt * sizeof(unsigned long long), c->stream));
  if (nacc) QV2_CUDA(c, cudaMemsetAsync(c->d_hist_acc, 0, nacc * sizeof(unsigned long long), c->stream));
  QV2_CUDA(c, cudaMemsetAsync(c->d_tickets, 0, 3 * nt * sizeof(uint32_t), c->stream));
  c->plan = std::move(plan);
  c->plan_key = std::move(key);
  c->plan_valid = true;
  return QV2_OK;
}

Launch launch_of(qv2_ctx* c) {
  Launch l; l.stream = c->stream; l.sm_count = c->sm_count; l.pdl = c->dependent_launch;
  return l;
}

CalibArgs calib_args(qv2_ctx* c, float* gmin, float* gmax, float* gabsmax, uint64_t* hist, float* clip,
                     float* step, float* inv, float* offset, uint64_t* nonfinite) {
  const size_t nt = c->plan.tensors.size();
  CalibArgs a;
  a.tensors = c->d_tensors;
  a.kmin = c->d_keys; a.kmax = c->d_keys + c->plan.total_groups;
  a.rslots = c->d_rslots; a.nf_acc = c->d_nf_acc; a.hist_acc = c->d_hist_acc;
  a.tickets = c->d_tickets; a.hist_tickets = c->d_tickets + nt;
  a.tensor_absmax = c->d_tensor_absmax;
  a.gmin = gmin; a.gmax = gmax; a.gabsmax = gabsmax; a.step = step; a.inv = inv; a.offset = offset;
  a.clip = clip;
  a.nonfinite = reinterpret_cast<unsigned long long*>(nonfinite);
  a.hist = reinterpret_cast<unsigned long long*>(hist);
  return a;
}

MetricsArgs metrics_args(qv2_ctx* c, const float* step, const float* inv, const float* offset, uint8_t* const* codes,
                         double* xe, double* sse, double* sig, double* mse, double* sqnr_db, double* cosine) {
  MetricsArgs a;
  a.tensors = c->d_tensors; a.step = step; a.inv = inv; a.offset = offset; a.codes = codes;
  a.partials = c->d_partials; a.partials_xe = xe;
  a.tickets = c->d_tickets + 2 * c->plan.tensors.size();
  a.sse = sse; a.sig = sig; a.mse = mse; a.sqnr_db = sqnr_db; a.cosine = cosine;
  return a;
}

// Range and histogram phases of one stage.
int run_calib_stage(qv2_ctx* c, const Stage& st, const CalibArgs& a) {
  const Launch l = launch_of(c);
  // a stage that folds in its streaming kernels is one launch per phase; otherwise the streaming
  // kernel (when the stage has tiles) and a fold kernel
  const uint64_t per_range = st.fused_fold ? 1 : (st.tile_end > st.tile_begin ? 2 : 1);
  const uint64_t per_hist = st.fused_fold ? 1 : (st.hist_end > st.hist_begin ? 2 : 1);
  QV2_CUDA(c, launch_range(l, st, c->plan.any_16bit, c->d_tiles, a));
  c->launches += per_range;
  if (st.any_percentile) {
    QV2_CUDA(c, launch_hist(l, st, c->plan.any_16bit, c->d_hist_tiles, a));
    c->launches += per_hist;
  }
  return QV2_OK;
}

int run_metrics_stage(qv2_ctx* c, const Stage& st, const MetricsArgs& a) {
  QV2_CUDA(c, launch_metrics(launch_of(c), st, c->plan.any_16bit, c->d_tiles, a));
  c->launches += st.fused_fold ? 1 : (st.tile_end > st.tile_begin ? 2 : 1);
  return QV2_OK;
}

// Per-group percentile clips (a separate, group-major pass; plans that have it are single-stage).
int run_group_percentile(qv2_ctx* c, uint32_t n, const CalibArgs& a, uint64_t* group_hist, float* group_clip) {
  const HostPlan& p = c->plan;
  const size_t n_ghist = p.ghist_owner.size();
  const Launch l = launch_of(c);
  int st;
  if (n_ghist) {
    unsigned long long* gh = reinterpret_cast<unsigned long long*>(group_hist);
    if (!gh) {
      if ((st = grow(c, &c->d_ghist, &c->cap_ghist, n_ghist * kBins)) != QV2_OK) return st;
      gh = c->d_ghist;
    }
    QV2_CUDA(c, cudaMemsetAsync(gh, 0, n_ghist * kBins * sizeof(uint64_t), c->stream));
    QV2_CUDA(c, launch_group_hist(l, c->caps.ghist, p.any_16bit, c->d_tensors, c->d_ghist_tiles,
                                  (uint32_t)p.ghist_tiles.size(), a.gabsmax, a.nonfinite, gh));
    QV2_CUDA(c, launch_group_clip_finalize(l, c->d_tensors, c->d_ghist_owner, (uint32_t)n_ghist, gh, a.nonfinite, a.gmin, a.gmax,
                                           a.gabsmax, group_clip, a.step, a.inv, a.offset));
    c->launches += p.ghist_tiles.empty() ? 1 : 2;
  }
  if (group_clip) {
    QV2_CUDA(c, launch_fill_group_clip(l, c->d_tensors, n, a.clip, group_clip));
    ++c->launches;
  }
  return QV2_OK;
}

// Makes the device table of code pointers current for this call.  The table is refilled from one
// of a few pinned areas; an area is reused only once the copy that read it has completed, which
// in steady state is long past, so the call does not wait.
int upload_codes(qv2_ctx* c, void* const* codes, const qv2_tensor_desc* descs, uint32_t n) {
  int st;
  if ((st = grow(c, &c->d_codes, &c->cap_codes, n, false)) != QV2_OK) return st;
  if (c->cap_h_codes < n) {
    if ((st = sync_stream(c)) != QV2_OK) return st;
    for (int i = 0; i < kCodeRing; ++i) {
      if (c->h_codes[i]) { QV2_CUDA(c, cudaFreeHost(c->h_codes[i])); c->h_codes[i] = nullptr; }
      if (!c->code_ev[i]) QV2_CUDA(c, cudaEventCreateWithFlags(&c->code_ev[i], cudaEventDisableTiming));
    }
    c->cap_h_codes = 0;
    const size_t want = (size_t)n + n / 4 + 16;
    for (int i = 0; i < kCodeRing; ++i) QV2_CUDA(c, cudaMallocHost((void**)&c->h_codes[i], want * sizeof(uint8_t*)));
    c->cap_h_codes = want;
  }
  const uint32_t k = c->code_next++ % kCodeRing;
  QV2_CUDA(c, cudaEventSynchronize(c->code_ev[k]));      // completed long ago unless calls pile up
  for (uint32_t t = 0; t < n; ++t)
    c->h_codes[k][t] = (descs[t].flags & QV2_STORE_CODES) ? (uint8_t*)codes[t] : nullptr;
  QV2_CUDA(c, cudaMemcpyAsync(c->d_codes, c->h_codes[k], (size_t)n * sizeof(uint8_t*), cudaMemcpyHostToDevice,
                              c->stream));
  QV2_CUDA(c, cudaEventRecord(c->code_ev[k], c->stream));
  return QV2_OK;
}

}  // namespace

extern "C" const char* qv2_status_string(int status) {
  switch (status) {
    case QV2_OK: return "QV2_OK";
    case QV2_ERR_ARG: return "QV2_ERR_ARG: invalid argument";
    case QV2_ERR_NULL: return "QV2_ERR_NULL: required pointer is NULL";
    case QV2_ERR_ALIGN: return "QV2_ERR_ALIGN: pointer is not sufficiently aligned";
    case QV2_ERR_SIZE: return "QV2_ERR_SIZE: size outside the supported range";
    case QV2_ERR_NONFINITE: return "QV2_ERR_NONFINITE: input holds NaN or Inf";
    case QV2_ERR_CUDA: return "QV2_ERR_CUDA: CUDA runtime call failed";
    case QV2_ERR_NOMEM: return "QV2_ERR_NOMEM: out of memory";
    case QV2_ERR_UNSUPPORTED: return "QV2_ERR_UNSUPPORTED: not implemented";
    default: return "QV2: unknown status";
  }
}

extern "C" int qv2_create(qv2_ctx** out, int device, void* stream) {
  if (!out) return QV2_ERR_NULL;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return QV2_ERR_CUDA;
  qv2_ctx* c = new (std::nothrow) qv2_ctx();
  if (!c) return QV2_ERR_NOMEM;
  c->device = device;
  c->stream = (cudaStream_t)stream;
  DeviceGuard guard(device);
  int sms = 0;
  cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaMalloc((void**)&c->d_rank, kRankScratchDoubles * sizeof(double));
  if (e != cudaSuccess) { delete c; return e == cudaErrorMemoryAllocation ? QV2_ERR_NOMEM : QV2_ERR_CUDA; }
  c->sm_count = sms > 0 ? sms : 1;
  // occupancy of each persistent kernel on THIS device (two contexts on different GPUs differ)
  c->caps.range = range_grid_cap(c->sm_count, false);
  c->caps.hist = hist_grid_cap(c->sm_count, false);
  c->caps.metrics = metrics_grid_cap(c->sm_count, false);
  c->caps.range_fused = range_grid_cap(c->sm_count, true);
  c->caps.hist_fused = hist_grid_cap(c->sm_count, true);
  c->caps.metrics_fused = metrics_grid_cap(c->sm_count, true);
  c->caps.ghist = group_hist_grid_cap(c->sm_count);
  c->caps.kl = kl_grid_cap(c->sm_count);
  const char* lg = std::getenv("QV2_LOG");
  c->log = lg && lg[0] == '1';
  *out = c;
  return QV2_OK;
}

extern "C" int qv2_destroy(qv2_ctx* c) {
  if (!c) return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  cudaStreamSynchronize(c->stream);
  cudaFree(c->d_tensors); cudaFree(c->d_tiles); cudaFree(c->d_hist_tiles); cudaFree(c->d_ghist_tiles);
  cudaFree(c->d_ghist_owner); cudaFree(c->d_ghist); cudaFree(c->d_partials); cudaFree(c->d_rslots);
  cudaFree(c->d_partials_xe); cudaFree(c->d_kl_hist); cudaFree(c->d_tensor_absmax); cudaFree(c->d_keys);
  cudaFree(c->d_nf_acc); cudaFree(c->d_hist_acc); cudaFree(c->d_tickets); cudaFree(c->d_codes);
  cudaFree(c->d_rank);
  if (c->h_pinned) cudaFreeHost(c->h_pinned);
  for (int i = 0; i < kCodeRing; ++i) {
    if (c->h_codes[i]) cudaFreeHost(c->h_codes[i]);
    if (c->code_ev[i]) cudaEventDestroy(c->code_ev[i]);
  }
  for (cudaEvent_t e : c->phase_ev)
    if (e) cudaEventDestroy(e);
  delete c;
  return QV2_OK;
}

extern "C" int qv2_last_cuda_error(const qv2_ctx* c) { return c ? c->last_cuda : 0; }
extern "C" uint64_t qv2_launch_count(const qv2_ctx* c) { return c ? c->launches : 0; }
extern "C" uint64_t qv2_sync_count(const qv2_ctx* c) { return c ? c->syncs : 0; }

extern "C" int qv2_set_schedule(qv2_ctx* c, uint32_t schedule, uint64_t chunk_bytes) {
  if (!c) return QV2_ERR_NULL;
  if (schedule > QV2_SCHEDULE_AUTO) return QV2_ERR_ARG;
  if (c->live_graphs) return QV2_ERR_UNSUPPORTED;     // a captured pass replays the schedule it was captured with
  c->schedule = schedule;
  c->chunk_bytes = chunk_bytes ? chunk_bytes : kDefaultChunkBytes;
  return QV2_OK;
}

extern "C" int qv2_set_fold_mode(qv2_ctx* c, uint32_t mode) {
  if (!c) return QV2_ERR_NULL;
  if (mode > QV2_FOLD_SEPARATE) return QV2_ERR_ARG;
  if (c->live_graphs) return QV2_ERR_UNSUPPORTED;
  c->fold_mode = mode;
  return QV2_OK;
}

extern "C" int qv2_set_dependent_launch(qv2_ctx* c, int on) {
  if (!c) return QV2_ERR_NULL;
  if (c->live_graphs) return QV2_ERR_UNSUPPORTED;     // a captured pass keeps the edges it was captured with
  c->dependent_launch = on != 0;
  return QV2_OK;
}

extern "C" int qv2_set_phase_timing(qv2_ctx* c, int on) {
  if (!c) return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  if (on)
    for (cudaEvent_t& e : c->phase_ev)
      if (!e) QV2_CUDA(c, cudaEventCreate(&e));
  c->phase_timing = on != 0;
  c->phase_marks_valid = false;
  return QV2_OK;
}

extern "C" int qv2_calibrate_phase_ms(qv2_ctx* c, float* range_ms, float* hist_ms) {
  if (!c || !range_ms || !hist_ms) return QV2_ERR_NULL;
  if (!c->phase_timing || !c->phase_marks_valid) return QV2_ERR_UNSUPPORTED;
  DeviceGuard guard(c->device);
  ++c->syncs;
  QV2_CUDA(c, cudaEventSynchronize(c->phase_ev[2]));
  QV2_CUDA(c, cudaEventElapsedTime(range_ms, c->phase_ev[0], c->phase_ev[1]));
  QV2_CUDA(c, cudaEventElapsedTime(hist_ms, c->phase_ev[1], c->phase_ev[2]));
  return QV2_OK;
}

extern "C" uint32_t qv2_stage_count(const qv2_ctx* c) {
  return (c && c->plan_valid) ? (uint32_t)c->plan.stages.size() : 0u;
}

namespace {

int calibrate_impl(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, float* gmin, float* gmax,
                   float* gabsmax, uint64_t* hist, float* clip, float* step, float* inv, float* offset,
                   uint64_t* nonfinite, uint64_t* group_hist, float* group_clip) {
  int st = ensure_plan(c, descs, n);
  if (st != QV2_OK) return st;
  const CalibArgs a = calib_args(c, gmin, gmax, gabsmax, hist, clip, step, inv, offset, nonfinite);
  if (c->phase_timing && c->plan.stages.size() == 1) {
    // measurement aid: the two phases as separate launches with an event between them
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    QV2_CUDA(c, cudaStreamIsCapturing(c->stream, &cap));
    if (cap == cudaStreamCaptureStatusNone) {
      const Stage& sg = c->plan.stages[0];
      const Launch l = launch_of(c);
      c->phase_marks_valid = false;
      QV2_CUDA(c, cudaEventRecord(c->phase_ev[0], c->stream));
      QV2_CUDA(c, launch_range(l, sg, c->plan.any_16bit, c->d_tiles, a));
      c->launches += sg.fused_fold ? 1 : (sg.tile_end > sg.tile_begin ? 2 : 1);
      QV2_CUDA(c, cudaEventRecord(c->phase_ev[1], c->stream));
      if (sg.any_percentile) {
        QV2_CUDA(c, launch_hist(l, sg, c->plan.any_16bit, c->d_hist_tiles, a));
        c->launches += sg.fused_fold ? 1 : (sg.hist_end > sg.hist_begin ? 2 : 1);
      }
      if ((st = run_group_percentile(c, n, a, group_hist, group_clip)) != QV2_OK) return st;
      QV2_CUDA(c, cudaEventRecord(c->phase_ev[2], c->stream));
      c->phase_marks_valid = true;
      return QV2_OK;
    }
  }
  for (const Stage& sg : c->plan.stages)
    if ((st = run_calib_stage(c, sg, a)) != QV2_OK) return st;
  return run_group_percentile(c, n, a, group_hist, group_clip);
}

int metrics_impl(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, const float* step, const float* inv,
                 const float* offset, void* const* codes, double* sse, double* sig, double* mse,
                 double* sqnr_db, double* cosine) {
  bool any_codes = false;
  if (codes)
    for (uint32_t t = 0; t < n && n <= 65535u; ++t)
      if ((descs[t].flags & QV2_STORE_CODES) && codes[t]) any_codes = true;
  int st = ensure_plan(c, descs, n);
  if (st != QV2_OK) return st;
  if (any_codes && (st = upload_codes(c, codes, descs, n)) != QV2_OK) return st;
  double* xe = nullptr;
  if (cosine) {                        // third slot array, only when the cosine is wanted
    const size_t need = c->plan.total_slots ? c->plan.total_slots : 1;
    if ((st = grow(c, &c->d_partials_xe, &c->cap_slots_xe, need, false)) != QV2_OK) return st;
    xe = c->d_partials_xe;
  }
  const MetricsArgs a = metrics_args(c, step, inv, offset, any_codes ? c->d_codes : nullptr, xe, sse, sig, mse,
                                     sqnr_db, cosine);
  for (const Stage& sg : c->plan.stages)
    if ((st = run_metrics_stage(c, sg, a)) != QV2_OK) return st;
  return QV2_OK;
}

}  // namespace

extern "C" int qv2_calibrate_ex(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, float* gmin,
                                float* gmax, float* gabsmax, uint64_t* hist, float* clip, float* step,
                                float* inv, float* offset, uint64_t* nonfinite, uint64_t* group_hist,
                                float* group_clip) {
  if (!c || !descs || !gmin || !gmax || !gabsmax || !clip || !step || !inv || !offset || !nonfinite)
    return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  TraceRange trace("qv2_calibrate");
  const uint64_t before = c->launches;
  const int st = calibrate_impl(c, descs, n, gmin, gmax, gabsmax, hist, clip, step, inv, offset, nonfinite,
                                group_hist, group_clip);
  log_call(c, "qv2_calibrate", n, before, st);
  return st;
}

extern "C" int qv2_calibrate(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, float* gmin,
                             float* gmax, float* gabsmax, uint64_t* hist, float* clip, float* step,
                             float* inv, float* offset, uint64_t* nonfinite) {
  return qv2_calibrate_ex(c, descs, n, gmin, gmax, gabsmax, hist, clip, step, inv, offset, nonfinite,
                          nullptr, nullptr);
}

extern "C" int qv2_quant_metrics_ex(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n,
                                    const float* step, const float* inv, const float* offset,
                                    void* const* codes, double* sse, double* sig, double* mse,
                                    double* sqnr_db, double* cosine) {
  if (!c || !descs || !step || !inv || !offset || !sse || !sig || !mse || !sqnr_db) return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  TraceRange trace("qv2_quant_metrics");
  const uint64_t before = c->launches;
  const int st = metrics_impl(c, descs, n, step, inv, offset, codes, sse, sig, mse, sqnr_db, cosine);
  log_call(c, "qv2_quant_metrics", n, before, st);
  return st;
}

extern "C" int qv2_quant_metrics(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n,
                                 const float* step, const float* inv, const float* offset,
                                 void* const* codes, double* sse, double* sig, double* mse,
                                 double* sqnr_db) {
  return qv2_quant_metrics_ex(c, descs, n, step, inv, offset, codes, sse, sig, mse, sqnr_db, nullptr);
}

extern "C" int qv2_kl_divergence(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, const float* step,
                                 const float* inv, const float* offset, const float* gabsmax, double* kl,
                                 uint64_t* hists) {
  if (!c || !descs || !step || !inv || !offset || !gabsmax || !kl) return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  TraceRange trace("qv2_kl_divergence");
  int st = ensure_plan(c, descs, n);
  if (st != QV2_OK) return st;
  const HostPlan& p = c->plan;
  unsigned long long* h = reinterpret_cast<unsigned long long*>(hists);
  const size_t cells = (size_t)n * 2 * QV2_KL_BINS;
  if (!h) {
    if ((st = grow(c, &c->d_kl_hist, &c->cap_kl_hist, cells, false)) != QV2_OK) return st;
    h = c->d_kl_hist;
  }
  QV2_CUDA(c, cudaMemsetAsync(h, 0, cells * sizeof(unsigned long long), c->stream));
  QV2_CUDA(c, launch_kl(launch_of(c), c->caps.kl, c->d_tensors, n, c->d_tiles, (uint32_t)p.tiles.size(), step, inv,
                        offset, gabsmax, c->d_tensor_absmax, h, kl));
  c->launches += p.tiles.empty() ? 2 : 3;
  return QV2_OK;
}

extern "C" int qv2_check_nonfinite(qv2_ctx* c, const uint64_t* nonfinite, uint32_t n, uint32_t* first_bad) {
  if (!c || !nonfinite) return QV2_ERR_NULL;
  if (n == 0 || n > 65535u) return QV2_ERR_SIZE;
  DeviceGuard guard(c->device);
  std::vector<uint64_t> host(n);
  QV2_CUDA(c, cudaMemcpyAsync(host.data(), nonfinite, (size_t)n * sizeof(uint64_t), cudaMemcpyDeviceToHost,
                              c->stream));
  if (int st = sync_stream(c)) return st;
  for (uint32_t t = 0; t < n; ++t)
    if (host[t]) { if (first_bad) *first_bad = t; return QV2_ERR_NONFINITE; }
  return QV2_OK;
}

extern "C" int qv2_fold_batchnorm(qv2_ctx* c, const float* w, const float* bias, const float* gamma,
                                  const float* beta, const float* mean, const float* var,
                                  uint64_t channels, uint64_t inner, float* w_out, float* bias_out) {
  if (!c || !gamma || !beta || !mean || !var) return QV2_ERR_NULL;
  if (channels && inner && (!w || !w_out)) return QV2_ERR_NULL;
  if (channels != 0 && inner > (1ull << 62) / channels) return QV2_ERR_SIZE;
  if ((((uintptr_t)w) | ((uintptr_t)w_out)) & 3u) return QV2_ERR_ALIGN;
  if (w != w_out && channels && inner) {        // in place is fine, a partial overlap is not
    const uintptr_t a0 = (uintptr_t)w, b0 = (uintptr_t)w_out, len = (uintptr_t)(channels * inner * sizeof(float));
    if (a0 < b0 + len && b0 < a0 + len) return QV2_ERR_ARG;
  }
  DeviceGuard guard(c->device);
  QV2_CUDA(c, launch_fold(launch_of(c), w, bias, gamma, beta, mean, var, channels, inner, w_out, bias_out));
  c->launches += (channels && inner ? (channels + 65534) / 65535 : 0) + (bias_out && channels ? 1 : 0);
  return QV2_OK;
}

extern "C" int qv2_rank_layers_ex(qv2_ctx* c, uint32_t n_layers, const double* sqnr_w,
                                  const double* mse_w, const double* sqnr_a, const double* mse_a,
                                  const uint64_t* macs, const double* pos, const uint32_t* fuse_group,
                                  const qv2_rank_cfg* cfg, uint32_t* order, uint8_t* keep_fp32,
                                  uint32_t* n_keep) {
  if (!c || !sqnr_w || !mse_w || !sqnr_a || !mse_a || !cfg || !order || !keep_fp32 || !n_keep)
    return QV2_ERR_NULL;
  if (n_layers == 0 || n_layers > kMaxRankLayers) return QV2_ERR_SIZE;
  if (cfg->select_mode > QV2_BY_BOPS_RATE) return QV2_ERR_ARG;
  if (cfg->select_mode == QV2_BY_BOPS_RATE && cfg->rate_permyriad > 10000u) return QV2_ERR_ARG;
  if (cfg->outlier_order > QV2_OUTLIERS_LITERAL) return QV2_ERR_ARG;
  DeviceGuard guard(c->device);
  TraceRange trace("qv2_rank_layers");
  QV2_CUDA(c, launch_rank(launch_of(c), n_layers, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, fuse_group,
                          *cfg, c->d_rank, order, keep_fp32, n_keep));
  ++c->launches;
  if (c->log) std::fprintf(stderr, "qv2: qv2_rank_layers layers=%u launches=1 status=0 (QV2_OK)\n", n_layers);
  return QV2_OK;
}

extern "C" int qv2_rank_layers(qv2_ctx* c, uint32_t n_layers, const double* sqnr_w,
                               const double* mse_w, const double* sqnr_a, const double* mse_a,
                               const uint64_t* macs, const double* pos, const qv2_rank_cfg* cfg,
                               uint32_t* order, uint8_t* keep_fp32, uint32_t* n_keep) {
  return qv2_rank_layers_ex(c, n_layers, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, nullptr, cfg, order,
                            keep_fp32, n_keep);
}

extern "C" int qv2_sweep_model(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n_tensors,
                               uint32_t n_layers, const uint64_t* macs, const double* pos,
                               const qv2_rank_cfg* cfg, const qv2_sweep_buffers* b) {
  if (!c || !descs || !cfg || !b) return QV2_ERR_NULL;
  if (n_layers == 0 || n_layers > kMaxRankLayers) return QV2_ERR_SIZE;
  if ((uint64_t)n_tensors < 2ull * n_layers) return QV2_ERR_ARG;
  if (!b->order || !b->keep_fp32 || !b->n_keep || !b->sse || !b->sig || !b->mse || !b->sqnr_db)
    return QV2_ERR_NULL;
  if (!b->gmin || !b->gmax || !b->gabsmax || !b->clip || !b->step || !b->inv || !b->offset || !b->nonfinite)
    return QV2_ERR_NULL;
  if (cfg->select_mode > QV2_BY_BOPS_RATE) return QV2_ERR_ARG;
  if (cfg->select_mode == QV2_BY_BOPS_RATE && cfg->rate_permyriad > 10000u) return QV2_ERR_ARG;
  DeviceGuard guard(c->device);
  int st = ensure_plan(c, descs, n_tensors);
  if (st != QV2_OK) return st;
  if (c->plan.stages.size() <= 1) {          // phase-major: the three calls of the contract, chained
    st = qv2_calibrate(c, descs, n_tensors, b->gmin, b->gmax, b->gabsmax, b->hist, b->clip, b->step,
                       b->inv, b->offset, b->nonfinite);
    if (st != QV2_OK) return st;
    st = qv2_quant_metrics(c, descs, n_tensors, b->step, b->inv, b->offset, nullptr, b->sse, b->sig,
                           b->mse, b->sqnr_db);
    if (st != QV2_OK) return st;
  } else {
    // L2-chunked: range -> histogram -> metrics stage by stage, so that the second and third read
    // of a stage's reference tensors hit L2
    TraceRange trace("qv2_sweep_model (L2-chunked)");
    const uint64_t before = c->launches;
    const CalibArgs ca = calib_args(c, b->gmin, b->gmax, b->gabsmax, b->hist, b->clip, b->step, b->inv,
                                    b->offset, b->nonfinite);
    const MetricsArgs ma = metrics_args(c, b->step, b->inv, b->offset, nullptr, nullptr, b->sse, b->sig,
                                        b->mse, b->sqnr_db, nullptr);
    for (const Stage& sg : c->plan.stages) {
      if ((st = run_calib_stage(c, sg, ca)) != QV2_OK) break;
      if ((st = run_metrics_stage(c, sg, ma)) != QV2_OK) break;
    }
    log_call(c, "qv2_sweep_model (L2-chunked calibrate+metrics)", n_tensors, before, st);
    if (st != QV2_OK) return st;
  }
  return qv2_rank_layers(c, n_layers, b->sqnr_db, b->mse, b->sqnr_db + n_layers, b->mse + n_layers,
                         macs, pos, cfg, b->order, b->keep_fp32, b->n_keep);
}

namespace {
inline uint64_t align256(uint64_t v) { return (v + 255u) & ~(uint64_t)255u; }
}

extern "C" uint64_t qv2_staging_bytes(const qv2_tensor_desc* descs, uint32_t n_tensors,
                                      uint32_t n_layers) {
  if (!descs) return 0;
  uint64_t total = 0;
  for (uint32_t t = 0; t < n_tensors; ++t) {
    const uint64_t esz = dtype_size((descs[t].flags & QV2_IN_MASK) >> 16);
    const uint64_t bytes = align256(descs[t].outer * descs[t].channels * descs[t].inner * esz);
    total += bytes;
    if (descs[t].y) total += bytes;
  }
  total += align256((uint64_t)n_layers * sizeof(uint64_t)) + align256((uint64_t)n_layers * sizeof(double));
  return total + 256;
}

extern "C" int qv2_sweep_model_host(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n_tensors,
                                    uint32_t n_layers, const uint64_t* macs, const double* pos,
                                    const qv2_rank_cfg* cfg, void* staging, uint64_t staging_bytes,
                                    const qv2_sweep_buffers* b, const qv2_host_results* out) {
  if (!c || !descs || !cfg || !staging || !b || !out) return QV2_ERR_NULL;
  if (!out->mse || !out->sqnr_db || !out->nonfinite || !out->order || !out->keep_fp32 || !out->n_keep)
    return QV2_ERR_NULL;
  if (n_tensors == 0 || n_tensors > 65535u) return QV2_ERR_SIZE;
  if (staging_bytes < qv2_staging_bytes(descs, n_tensors, n_layers)) return QV2_ERR_SIZE;
  if ((uintptr_t)staging & 255u) return QV2_ERR_ALIGN;
  DeviceGuard guard(c->device);
  std::vector<qv2_tensor_desc> dd(descs, descs + n_tensors);
  uint8_t* base = (uint8_t*)staging;
  uint64_t off = 0;
  for (uint32_t t = 0; t < n_tensors; ++t) {
    if (dd[t].flags & QV2_STORE_CODES) return QV2_ERR_UNSUPPORTED;
    const uint64_t bytes = descs[t].outer * descs[t].channels * descs[t].inner *
                           dtype_size((descs[t].flags & QV2_IN_MASK) >> 16);
    if (bytes && !descs[t].x) return QV2_ERR_NULL;
    dd[t].x = (const float*)(base + off);
    if (bytes) QV2_CUDA(c, cudaMemcpyAsync(base + off, descs[t].x, bytes, cudaMemcpyHostToDevice, c->stream));
    off += align256(bytes);
    if (descs[t].y) {
      dd[t].y = (const float*)(base + off);
      if (bytes) QV2_CUDA(c, cudaMemcpyAsync(base + off, descs[t].y, bytes, cudaMemcpyHostToDevice, c->stream));
      off += align256(bytes);
    }
  }
  const uint64_t* d_macs = nullptr;
  const double* d_pos = nullptr;
  if (macs) {
    d_macs = (const uint64_t*)(base + off);
    QV2_CUDA(c, cudaMemcpyAsync(base + off, macs, (size_t)n_layers * sizeof(uint64_t), cudaMemcpyHostToDevice, c->stream));
  }
  off += align256((uint64_t)n_layers * sizeof(uint64_t));
  if (pos) {
    d_pos = (const double*)(base + off);
    QV2_CUDA(c, cudaMemcpyAsync(base + off, pos, (size_t)n_layers * sizeof(double), cudaMemcpyHostToDevice, c->stream));
  }
  int st = qv2_sweep_model(c, dd.data(), n_tensors, n_layers, d_macs, d_pos, cfg, b);
  if (st != QV2_OK) return st;
  const cudaMemcpyKind d2h = cudaMemcpyDeviceToHost;
  QV2_CUDA(c, cudaMemcpyAsync(out->mse, b->mse, (size_t)n_tensors * sizeof(double), d2h, c->stream));
  QV2_CUDA(c, cudaMemcpyAsync(out->sqnr_db, b->sqnr_db, (size_t)n_tensors * sizeof(double), d2h, c->stream));
  QV2_CUDA(c, cudaMemcpyAsync(out->nonfinite, b->nonfinite, (size_t)n_tensors * sizeof(uint64_t), d2h, c->stream));
  QV2_CUDA(c, cudaMemcpyAsync(out->order, b->order, (size_t)n_layers * sizeof(uint32_t), d2h, c->stream));
  QV2_CUDA(c, cudaMemcpyAsync(out->keep_fp32, b->keep_fp32, (size_t)n_layers, d2h, c->stream));
  QV2_CUDA(c, cudaMemcpyAsync(out->n_keep, b->n_keep, sizeof(uint32_t), d2h, c->stream));
  if (int sst = sync_stream(c)) return sst;
  for (uint32_t t = 0; t < n_tensors; ++t)
    if (out->nonfinite[t]) return QV2_ERR_NONFINITE;
  return QV2_OK;
}

// ------------------------------------------------------------------------------------------------
// A whole pass captured once in a CUDA graph and replayed with one launch.
struct qv2_graph {
  qv2_ctx* ctx = nullptr;
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  uint64_t launches_per_replay = 0;
};

extern "C" int qv2_sweep_graph_create(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n_tensors,
                                      uint32_t n_layers, const uint64_t* macs, const double* pos,
                                      const qv2_rank_cfg* cfg, const qv2_sweep_buffers* bufs,
                                      qv2_graph** out) {
  if (!out) return QV2_ERR_NULL;
  *out = nullptr;
  if (!c) return QV2_ERR_NULL;
  if (c->stream == nullptr || c->stream == cudaStreamLegacy) return QV2_ERR_UNSUPPORTED;  // cannot be captured
  DeviceGuard guard(c->device);
  // First an ordinary pass: validates the arguments, makes the tile tables resident and sizes
  // every scratch buffer, so that the captured pass allocates and uploads nothing.
  const uint64_t before = c->launches;
  int st = qv2_sweep_model(c, descs, n_tensors, n_layers, macs, pos, cfg, bufs);
  if (st != QV2_OK) return st;
  const uint64_t per_pass = c->launches - before;
  if ((st = sync_stream(c)) != QV2_OK) return st;
  qv2_graph* g = new (std::nothrow) qv2_graph();
  if (!g) return QV2_ERR_NOMEM;
  g->ctx = c; g->launches_per_replay = per_pass;
  cudaError_t e = cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal);
  if (e != cudaSuccess) { delete g; return cuda_fail(c, e); }
  st = qv2_sweep_model(c, descs, n_tensors, n_layers, macs, pos, cfg, bufs);
  c->launches -= (st == QV2_OK) ? per_pass : 0;        // captured, not executed
  e = cudaStreamEndCapture(c->stream, &g->graph);
  if (st != QV2_OK || e != cudaSuccess || !g->graph) {
    if (g->graph) cudaGraphDestroy(g->graph);
    delete g;
    return st != QV2_OK ? st : cuda_fail(c, e != cudaSuccess ? e : cudaErrorUnknown);
  }
  e = cudaGraphInstantiate(&g->exec, g->graph, 0);
  if (e != cudaSuccess) { cudaGraphDestroy(g->graph); delete g; return cuda_fail(c, e); }
  ++c->live_graphs;                 // from now on the plan and its scratch stay where they are
  *out = g;
  return QV2_OK;
}

extern "C" int qv2_sweep_graph_launch(qv2_graph* g) {
  if (!g || !g->ctx || !g->exec) return QV2_ERR_NULL;
  DeviceGuard guard(g->ctx->device);
  QV2_CUDA(g->ctx, cudaGraphLaunch(g->exec, g->ctx->stream));
  g->ctx->launches += g->launches_per_replay;
  return QV2_OK;
}

extern "C" int qv2_sweep_graph_destroy(qv2_graph* g) {
  if (!g) return QV2_ERR_NULL;
  if (g->ctx) {
    DeviceGuard guard(g->ctx->device);
    cudaStreamSynchronize(g->ctx->stream);
    if (g->ctx->live_graphs) --g->ctx->live_graphs;
  }
  if (g->exec) cudaGraphExecDestroy(g->exec);
  if (g->graph) cudaGraphDestroy(g->graph);
  delete g;
  return QV2_OK;
}

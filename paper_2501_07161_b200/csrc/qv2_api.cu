// C-ABI layer: context, scratch management, plan caching and the call sequences of the public
// entry points declared in include/qv2.h.
#include <cstdlib>
#include <cstring>
#include <new>

#include "qv2_common.cuh"

using namespace qv2;

struct qv2_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  int sm_count = 1;
  uint32_t metrics_cap = 1;   // largest useful grid of the metrics kernel on this device
  uint32_t range_cap = 1;     // the same for the range kernel
  int last_cuda = 0;
  uint64_t launches = 0;

  // cached plan: rebuilt only when the descriptor bytes (or code pointers) change
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
  unsigned long long* d_hist = nullptr; size_t cap_hist = 0;   // used when the caller passes no hist
  double* d_rank = nullptr;                                    // 2 * kMaxRankLayers doubles
  // pinned host staging for the plan upload
  uint8_t* h_pinned = nullptr;    size_t cap_pinned = 0;
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

int cuda_fail(qv2_ctx* c, cudaError_t e) {
  c->last_cuda = (int)e;
  return e == cudaErrorMemoryAllocation ? QV2_ERR_NOMEM : QV2_ERR_CUDA;
}

#define QV2_CUDA(c, expr)                              \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) return cuda_fail((c), e__);\
  } while (0)

template <class T>
int grow(qv2_ctx* c, T** p, size_t* cap, size_t need) {
  if (need <= *cap) return QV2_OK;
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

int ensure_plan_checked(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, void* const* codes);

// Makes ctx->plan describe (descs, codes) and resident on the device.
int ensure_plan(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, void* const* codes) {
  try {
    return ensure_plan_checked(c, descs, n, codes);
  } catch (const std::bad_alloc&) {          // host tables did not fit: nothing unwinds through the C ABI
    c->plan_valid = false;
    return QV2_ERR_NOMEM;
  }
}

int ensure_plan_checked(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, void* const* codes) {
  if (!descs) return QV2_ERR_NULL;
  if (n == 0 || n > 65535u) return QV2_ERR_SIZE;
  const size_t dbytes = (size_t)n * sizeof(qv2_tensor_desc);
  const size_t cbytes = codes ? (size_t)n * sizeof(void*) : 0;
  std::vector<uint8_t> key(dbytes + cbytes + 1);
  std::memcpy(key.data(), descs, dbytes);
  if (codes) std::memcpy(key.data() + dbytes, codes, cbytes);
  key[dbytes + cbytes] = codes ? 1 : 0;
  if (c->plan_valid && key == c->plan_key) return QV2_OK;

  HostPlan plan;
  int st = build_plan(descs, n, codes, c->metrics_cap, c->range_cap, &plan);
  if (st != QV2_OK) return st;
  // The previous upload may still be reading the pinned buffer, and buffers may be reallocated.
  QV2_CUDA(c, cudaStreamSynchronize(c->stream));
  c->plan_valid = false;
  const size_t nt = plan.tensors.size(), ntl = plan.tiles.size(), nh = plan.hist_tiles.size();
  if ((st = grow(c, &c->d_tensors, &c->cap_tensors, nt)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_tiles, &c->cap_tiles, ntl ? ntl : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_hist_tiles, &c->cap_hist_tiles, nh ? nh : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_partials, &c->cap_slots, plan.total_slots ? plan.total_slots : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_rslots, &c->cap_rslots, plan.total_rslots ? plan.total_rslots : 1)) != QV2_OK) return st;
  if ((st = grow(c, &c->d_tensor_absmax, &c->cap_absmax, nt)) != QV2_OK) return st;
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
  c->plan = std::move(plan);
  c->plan_key = std::move(key);
  c->plan_valid = true;
  return QV2_OK;
}

Launch launch_of(qv2_ctx* c) {
  Launch l; l.stream = c->stream; l.sm_count = c->sm_count;
  return l;
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
  c->metrics_cap = metrics_grid_cap(c->sm_count);
  c->range_cap = range_grid_cap(c->sm_count);
  *out = c;
  return QV2_OK;
}

extern "C" int qv2_destroy(qv2_ctx* c) {
  if (!c) return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  cudaStreamSynchronize(c->stream);
  cudaFree(c->d_tensors); cudaFree(c->d_tiles); cudaFree(c->d_hist_tiles); cudaFree(c->d_ghist_tiles); cudaFree(c->d_ghist_owner); cudaFree(c->d_ghist); cudaFree(c->d_partials); cudaFree(c->d_rslots); cudaFree(c->d_partials_xe); cudaFree(c->d_kl_hist);
  cudaFree(c->d_tensor_absmax); cudaFree(c->d_hist); cudaFree(c->d_rank);
  if (c->h_pinned) cudaFreeHost(c->h_pinned);
  delete c;
  return QV2_OK;
}

extern "C" int qv2_last_cuda_error(const qv2_ctx* c) { return c ? c->last_cuda : 0; }
extern "C" uint64_t qv2_launch_count(const qv2_ctx* c) { return c ? c->launches : 0; }

extern "C" int qv2_calibrate_ex(qv2_ctx* c, const qv2_tensor_desc* descs, uint32_t n, float* gmin,
                                float* gmax, float* gabsmax, uint64_t* hist, float* clip, float* step,
                                float* inv, float* offset, uint64_t* nonfinite, uint64_t* group_hist,
                                float* group_clip) {
  if (!c || !descs || !gmin || !gmax || !gabsmax || !clip || !step || !inv || !offset || !nonfinite)
    return QV2_ERR_NULL;
  DeviceGuard guard(c->device);
  int st = ensure_plan(c, descs, n, nullptr);
  if (st != QV2_OK) return st;
  const HostPlan& p = c->plan;
  unsigned long long* h = reinterpret_cast<unsigned long long*>(hist);
  if (!h && p.any_percentile) {
    if ((st = grow(c, &c->d_hist, &c->cap_hist, (size_t)n * kBins)) != QV2_OK) return st;
    h = c->d_hist;
  }
  const size_t n_ghist = p.ghist_owner.size();
  unsigned long long* gh = reinterpret_cast<unsigned long long*>(group_hist);
  if (!gh && n_ghist) {
    if ((st = grow(c, &c->d_ghist, &c->cap_ghist, n_ghist * kBins)) != QV2_OK) return st;
    gh = c->d_ghist;
  }
  const Launch l = launch_of(c);
  const size_t G = (size_t)p.total_groups;
  QV2_CUDA(c, launch_calib_init(l, reinterpret_cast<uint32_t*>(gmin), reinterpret_cast<uint32_t*>(gmax), G,
                                reinterpret_cast<unsigned long long*>(nonfinite), n, h, h ? (size_t)n * kBins : 0));
  ++c->launches;
  if (n_ghist) QV2_CUDA(c, cudaMemsetAsync(gh, 0, n_ghist * kBins * sizeof(uint64_t), c->stream));
  if (!p.tiles.empty()) {
    QV2_CUDA(c, launch_range(l, p.range_grid, p.any_16bit, c->d_tensors, c->d_tiles, (uint32_t)p.tiles.size(),
                             reinterpret_cast<uint32_t*>(gmin), reinterpret_cast<uint32_t*>(gmax),
                             c->d_rslots, reinterpret_cast<unsigned long long*>(nonfinite)));
    ++c->launches;
  }
  QV2_CUDA(c, launch_range_finalize(l, c->d_tensors, n, c->d_rslots, gmin, gmax, gabsmax, step, inv, offset,
                                    c->d_tensor_absmax, clip));
  ++c->launches;
  if (!p.hist_tiles.empty()) {
    QV2_CUDA(c, launch_hist(l, p.any_16bit, c->d_tensors, c->d_hist_tiles, (uint32_t)p.hist_tiles.size(),
                            c->d_tensor_absmax, reinterpret_cast<unsigned long long*>(nonfinite), h));
    ++c->launches;
  }
  if (p.any_percentile) {              // clip[t] of the other tensors is already the absmax
    QV2_CUDA(c, launch_clip_finalize(l, c->d_tensors, n, h, c->d_tensor_absmax, gmin, gmax, gabsmax,
                                     clip, step, inv, offset));
    ++c->launches;
  }
  if (n_ghist) {
    QV2_CUDA(c, launch_group_hist(l, p.any_16bit, c->d_tensors, c->d_ghist_tiles, (uint32_t)p.ghist_tiles.size(),
                                  gabsmax, reinterpret_cast<unsigned long long*>(nonfinite), gh));
    QV2_CUDA(c, launch_group_clip_finalize(l, c->d_tensors, c->d_ghist_owner, (uint32_t)n_ghist, gh, gmin, gmax,
                                           gabsmax, group_clip, step, inv, offset));
    c->launches += p.ghist_tiles.empty() ? 1 : 2;
  }
  if (group_clip) {
    QV2_CUDA(c, launch_fill_group_clip(l, c->d_tensors, n, clip, group_clip));
    ++c->launches;
  }
  return QV2_OK;
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
  bool any_codes = false;
  if (codes)
    for (uint32_t t = 0; t < n && n <= 65535u; ++t)
      if ((descs[t].flags & QV2_STORE_CODES) && codes[t]) any_codes = true;
  int st = ensure_plan(c, descs, n, any_codes ? codes : nullptr);
  if (st != QV2_OK) return st;
  const HostPlan& p = c->plan;
  double* xe = nullptr;
  if (cosine) {                        // third slot array, only when the cosine is wanted
    if ((st = grow(c, &c->d_partials_xe, &c->cap_slots_xe, p.total_slots ? p.total_slots : 1)) != QV2_OK)
      return st;
    xe = c->d_partials_xe;
  }
  const Launch l = launch_of(c);
  if (!p.tiles.empty()) {
    QV2_CUDA(c, launch_metrics(l, p.metrics_grid, p.any_16bit, c->d_tensors, c->d_tiles, (uint32_t)p.tiles.size(), step, inv,
                               offset, c->d_partials, xe));
    ++c->launches;
  }
  QV2_CUDA(c, launch_metrics_finalize(l, c->d_tensors, n, c->d_partials, xe, sse, sig, mse, sqnr_db, cosine));
  ++c->launches;
  return QV2_OK;
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
  int st = ensure_plan(c, descs, n, nullptr);
  if (st != QV2_OK) return st;
  const HostPlan& p = c->plan;
  unsigned long long* h = reinterpret_cast<unsigned long long*>(hists);
  const size_t cells = (size_t)n * 2 * QV2_KL_BINS;
  if (!h) {
    if ((st = grow(c, &c->d_kl_hist, &c->cap_kl_hist, cells)) != QV2_OK) return st;
    h = c->d_kl_hist;
  }
  QV2_CUDA(c, cudaMemsetAsync(h, 0, cells * sizeof(unsigned long long), c->stream));
  QV2_CUDA(c, launch_kl(launch_of(c), c->d_tensors, n, c->d_tiles, (uint32_t)p.tiles.size(), step, inv,
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
  QV2_CUDA(c, cudaStreamSynchronize(c->stream));
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
  DeviceGuard guard(c->device);
  QV2_CUDA(c, launch_rank(launch_of(c), n_layers, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, fuse_group,
                          *cfg, c->d_rank, order, keep_fp32, n_keep));
  ++c->launches;
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
  if (cfg->select_mode > QV2_BY_BOPS_RATE) return QV2_ERR_ARG;
  if (cfg->select_mode == QV2_BY_BOPS_RATE && cfg->rate_permyriad > 10000u) return QV2_ERR_ARG;
  int st = qv2_calibrate(c, descs, n_tensors, b->gmin, b->gmax, b->gabsmax, b->hist, b->clip, b->step,
                         b->inv, b->offset, b->nonfinite);
  if (st != QV2_OK) return st;
  st = qv2_quant_metrics(c, descs, n_tensors, b->step, b->inv, b->offset, nullptr, b->sse, b->sig,
                         b->mse, b->sqnr_db);
  if (st != QV2_OK) return st;
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
  QV2_CUDA(c, cudaStreamSynchronize(c->stream));
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
  QV2_CUDA(c, cudaStreamSynchronize(c->stream));
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
  if (g->ctx) { DeviceGuard guard(g->ctx->device); cudaStreamSynchronize(g->ctx->stream); }
  if (g->exec) cudaGraphExecDestroy(g->exec);
  if (g->graph) cudaGraphDestroy(g->graph);
  delete g;
  return QV2_OK;
}

// Sensitivity list and mixed-precision layer set (Algorithm 2: CalculateSQNRdeltas,
// CalculateAverage, RankLayersBySensitivity; SQNR delta of Eq. 16; BOPs-reduction rate of Eq. 17).
//
// A model has tens of layers, so one CTA does everything.  Every binary64 operation is issued
// through an explicit round-to-nearest intrinsic so that no multiply-add is contracted and the
// result is a bit-exact function of the inputs.
#include "qv2_device.cuh"

namespace qv2 {

namespace {

__device__ __forceinline__ double clamp_cap(double v, double cap) {
  if (v > cap) return cap;
  if (v < -cap) return -cap;
  return v;
}

__global__ void __launch_bounds__(256)
rank_kernel(uint32_t n, const double* __restrict__ sqnr_w, const double* __restrict__ mse_w,
            const double* __restrict__ sqnr_a, const double* __restrict__ mse_a,
            const uint64_t* __restrict__ macs, const double* __restrict__ pos,
            const uint32_t* __restrict__ fuse_group, qv2_rank_cfg cfg, double* score, double* severity,
            uint32_t* place, uint32_t* best, uint32_t* order, uint8_t* keep, uint32_t* n_keep) {
  // Models have tens of layers: up to kStage layers the serial parts below run out of shared
  // memory instead of paying a global-memory latency per step.
  constexpr uint32_t kStage = 1024;
  __shared__ double mean_s[2];
  __shared__ double st_a[kStage], st_b[kStage];
  __shared__ unsigned long long st_macs[kStage];
  __shared__ uint32_t st_order[kStage], st_fg[kStage];
  constexpr uint32_t kNoGroup = QV2_NO_GROUP;
  const uint32_t tid = threadIdx.x;
  const bool staged = n <= kStage;
  const double inf = __longlong_as_double(0x7ff0000000000000ll);
  if (staged) {
    for (uint32_t i = tid; i < n; i += blockDim.x) {
      st_a[i] = mse_w[i]; st_b[i] = mse_a[i];
      st_macs[i] = macs ? macs[i] : 1ull;
      st_fg[i] = fuse_group ? fuse_group[i] : kNoGroup;
    }
    __syncthreads();
  }
  if (tid == 0) {                      // means: sums in layer order, as the definition states
    double sw = 0.0, sa = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
      sw = __dadd_rn(sw, staged ? st_a[i] : mse_w[i]);
      sa = __dadd_rn(sa, staged ? st_b[i] : mse_a[i]);
    }
    mean_s[0] = __ddiv_rn(sw, (double)n);
    mean_s[1] = __ddiv_rn(sa, (double)n);
  }
  __syncthreads();
  const double mean_w = mean_s[0], mean_a = mean_s[1], cap = cfg.sqnr_cap_db;
  for (uint32_t i = tid; i < n; i += blockDim.x) {
    double dw = 0.0, da = 0.0;
    if (i > 0) {
      const double den = pos ? __dsub_rn(pos[i], pos[i - 1]) : 1.0;
      dw = __ddiv_rn(__dsub_rn(clamp_cap(sqnr_w[i], cap), clamp_cap(sqnr_w[i - 1], cap)), den);
      da = __ddiv_rn(__dsub_rn(clamp_cap(sqnr_a[i], cap), clamp_cap(sqnr_a[i - 1], cap)), den);
    }
    double sc = __dadd_rn(__dmul_rn(cfg.w_gain, dw), __dmul_rn(cfg.a_gain, da));
    if (sc != sc) sc = inf;
    const double rw = mean_w > 0.0 ? __ddiv_rn(mse_w[i], mean_w) : 0.0;
    const double ra = mean_a > 0.0 ? __ddiv_rn(mse_a[i], mean_a) : 0.0;
    double sv = rw > ra ? rw : ra;
    if (sv != sv) sv = 0.0;
    score[i] = sc; severity[i] = sv; keep[i] = 0;
  }
  __syncthreads();
  // Position of layer i = number of layers that come before it: all MSE outliers precede the
  // rest; outliers by descending severity, the rest by ascending score, ties by layer index.
  const double fac = cfg.mse_factor;
  for (uint32_t i = tid; i < n; i += blockDim.x) {
    const double si = score[i], vi = severity[i];
    const bool out_i = vi > fac;
    uint32_t rank = 0;
    for (uint32_t j = 0; j < n; ++j) {
      const double vj = severity[j];
      const bool out_j = vj > fac;
      if (out_i) {
        if (out_j && (vj > vi || (vj == vi && j < i))) ++rank;
      } else {
        if (out_j) ++rank;
        else {
          const double sj = score[j];
          if (sj < si || (sj == si && j < i)) ++rank;
        }
      }
    }
    order[rank] = i;
    place[i] = rank;
  }
  __syncthreads();
  if (fuse_group) {
    // Fusion groups: every member moves to the place of the group's best-ranked member and the
    // members stand there in layer order.  Places of different groups differ, so sorting by
    // (best place of my group, layer index) yields exactly that list.
    for (uint32_t i = tid; i < n; i += blockDim.x) {
      const uint32_t g = fuse_group[i];
      uint32_t b = place[i];
      if (g != kNoGroup)
        for (uint32_t j = 0; j < n; ++j)
          if (fuse_group[j] == g) b = min(b, place[j]);
      best[i] = b;
    }
    __syncthreads();
    for (uint32_t i = tid; i < n; i += blockDim.x) {
      const uint32_t bi = best[i];
      uint32_t rank = 0;
      for (uint32_t j = 0; j < n; ++j) {
        const uint32_t bj = best[j];
        if (bj < bi || (bj == bi && j < i)) ++rank;
      }
      order[rank] = i;
    }
    __syncthreads();
  }
  if (staged) {
    for (uint32_t i = tid; i < n; i += blockDim.x) st_order[i] = order[i];
    __syncthreads();
  }
  if (tid == 0) {
    // The FP32-kept prefix grows one whole fusion group at a time (a layer without a group is a
    // group of one): by count while it still fits, by rate while the rate still holds.
    auto ord = [&](uint32_t j) { return staged ? st_order[j] : order[j]; };
    auto grp = [&](uint32_t l) { return staged ? st_fg[l] : (fuse_group ? fuse_group[l] : kNoGroup); };
    auto mac = [&](uint32_t l) { return staged ? st_macs[l] : (macs ? macs[l] : 1ull); };
    unsigned __int128 total = 0, kept = 0;
    if (cfg.select_mode != QV2_BY_COUNT)
      for (uint32_t i = 0; i < n; ++i) total += mac(i);
    uint32_t nk = 0, j = 0;
    while (j < n) {
      const uint32_t g = grp(ord(j));
      uint32_t e = j + 1;
      if (g != kNoGroup) while (e < n && grp(ord(e)) == g) ++e;
      if (cfg.select_mode == QV2_BY_COUNT) {
        if (e <= cfg.keep_count) nk = e; else break;
      } else {
        unsigned __int128 m = 0;
        for (uint32_t k = j; k < e; ++k) m += mac(ord(k));
        const unsigned __int128 quantized = total - (kept + m);
        if (quantized * 10000u >= (unsigned __int128)cfg.rate_permyriad * total) { kept += m; nk = e; }
        else break;
      }
      j = e;
    }
    for (uint32_t k = 0; k < nk; ++k) keep[ord(k)] = 1;
    *n_keep = nk;
  }
}

}  // namespace

cudaError_t launch_rank(const Launch& l, uint32_t n, const double* sqnr_w, const double* mse_w,
                        const double* sqnr_a, const double* mse_a, const uint64_t* macs,
                        const double* pos, const uint32_t* fuse_group, qv2_rank_cfg cfg, double* scratch,
                        uint32_t* order, uint8_t* keep, uint32_t* n_keep) {
  // scratch: kMaxRankLayers doubles each for score and severity, then two uint32 arrays
  uint32_t* place = reinterpret_cast<uint32_t*>(scratch + 2 * (size_t)kMaxRankLayers);
  rank_kernel<<<1, 256, 0, l.stream>>>(n, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, fuse_group, cfg,
                                       scratch, scratch + kMaxRankLayers, place, place + kMaxRankLayers,
                                       order, keep, n_keep);
  return cudaGetLastError();
}

}  // namespace qv2

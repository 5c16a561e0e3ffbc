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
  allow_dependents();
  dependency_wait();
  // Models have tens of layers: up to kStage layers every input and every intermediate lives in
  // shared memory, so the phases below cost one trip to global memory at the start and one at the
  // end instead of one per phase.  Larger n runs the same code on the global arrays.
  constexpr uint32_t kStage = 512;
  __shared__ double mean_s[2];
  __shared__ double s_mw[kStage], s_ma[kStage], s_sw[kStage], s_sa[kStage], s_pos[kStage], s_score[kStage],
      s_sev[kStage];
  __shared__ unsigned long long s_macs[kStage], s_mlist[kStage];
  __shared__ uint32_t s_fg[kStage], s_place[kStage], s_best[kStage], s_order[kStage];
  __shared__ uint8_t s_keep[kStage];
  constexpr uint32_t kNoGroup = QV2_NO_GROUP;
  const uint32_t tid = threadIdx.x;
  const bool staged = n <= kStage;
  const double inf = __longlong_as_double(0x7ff0000000000000ll);
  // the arrays the phases work on: shared copies when staged, the global ones otherwise
  const double *mw = mse_w, *ma = mse_a, *sw = sqnr_w, *sa = sqnr_a, *ps = pos;
  const unsigned long long* mc = reinterpret_cast<const unsigned long long*>(macs);
  const uint32_t* fg = fuse_group;
  double *sc = score, *sv = severity;
  uint32_t *pl = place, *bs = best, *od = order;
  uint8_t* kp = keep;
  if (staged) {
    for (uint32_t i = tid; i < n; i += blockDim.x) {
      s_mw[i] = mse_w[i]; s_ma[i] = mse_a[i]; s_sw[i] = sqnr_w[i]; s_sa[i] = sqnr_a[i];
      if (pos) s_pos[i] = pos[i];
      if (macs) s_macs[i] = macs[i];
      if (fuse_group) s_fg[i] = fuse_group[i];
    }
    mw = s_mw; ma = s_ma; sw = s_sw; sa = s_sa;
    if (pos) ps = s_pos;
    if (macs) mc = s_macs;
    if (fuse_group) fg = s_fg;
    sc = s_score; sv = s_sev; pl = s_place; bs = s_best; od = s_order; kp = s_keep;
    __syncthreads();
  }
  if (tid == 0 || tid == 32) {         // means: sums in layer order, as the definition states; one warp per list
    const double* m = tid == 0 ? mw : ma;
    double a = 0.0;
#pragma unroll 8
    for (uint32_t i = 0; i < n; ++i) a = __dadd_rn(a, m[i]);      // the loads run ahead of the chain of additions
    mean_s[tid == 0 ? 0 : 1] = __ddiv_rn(a, (double)n);
  }
  __syncthreads();
  const double mean_w = mean_s[0], mean_a = mean_s[1], cap = cfg.sqnr_cap_db;
  for (uint32_t i = tid; i < n; i += blockDim.x) {
    double dw = 0.0, da = 0.0;
    if (i > 0) {
      dw = __dsub_rn(clamp_cap(sw[i], cap), clamp_cap(sw[i - 1], cap));
      da = __dsub_rn(clamp_cap(sa[i], cap), clamp_cap(sa[i - 1], cap));
      if (ps) {                          // default positions 0,1,2,...: a division by 1 changes nothing
        const double den = __dsub_rn(ps[i], ps[i - 1]);
        dw = __ddiv_rn(dw, den);
        da = __ddiv_rn(da, den);
      }
    }
    double s = __dadd_rn(__dmul_rn(cfg.w_gain, dw), __dmul_rn(cfg.a_gain, da));
    if (s != s) s = inf;
    const double rw = mean_w > 0.0 ? __ddiv_rn(mw[i], mean_w) : 0.0;
    const double ra = mean_a > 0.0 ? __ddiv_rn(ma[i], mean_a) : 0.0;
    double v = rw > ra ? rw : ra;
    if (v != v) v = 0.0;
    sc[i] = s; sv[i] = v; kp[i] = 0;
  }
  __syncthreads();
  // Position of layer i = number of layers that come before it: all MSE outliers precede the
  // rest; outliers by descending severity (or, in the literal reading of the pseudo-code, where
  // each outlier is put at the head of the list when the layer loop meets it, in reverse layer
  // order), the rest by ascending score, ties by layer index.
  const double fac = cfg.mse_factor;
  const bool literal = cfg.outlier_order == QV2_OUTLIERS_LITERAL;
  // The n*n comparisons are spread over the whole block: with n <= blockDim/2 several threads share
  // a layer (thread p of a layer takes every parts-th j) and add their counts in `place`.
  const uint32_t parts = n <= blockDim.x / 2 ? blockDim.x / n : 1u;
  if (parts > 1) {
    for (uint32_t i = tid; i < n; i += blockDim.x) pl[i] = 0;
    __syncthreads();
  }
  for (uint32_t w = tid; w < n * parts; w += blockDim.x) {
    const uint32_t i = parts > 1 ? w % n : w, part = parts > 1 ? w / n : 0u;
    const double si = sc[i], vi = sv[i];
    const bool out_i = vi > fac;
    uint32_t rank = 0;
    if (out_i) {
#pragma unroll 4
      for (uint32_t j = part; j < n; j += parts) {
        const double vj = sv[j];
        const bool before = literal ? j > i : (vj > vi) | ((vj == vi) & (j < i));
        rank += (uint32_t)((vj > fac) & before);
      }
    } else {
#pragma unroll 4
      for (uint32_t j = part; j < n; j += parts) {
        const double vj = sv[j], sj = sc[j];
        rank += (uint32_t)((vj > fac) | (sj < si) | ((sj == si) & (j < i)));
      }
    }
    if (parts > 1) atomicAdd(pl + i, rank);
    else { od[rank] = i; pl[i] = rank; }
  }
  __syncthreads();
  if (parts > 1) {
    for (uint32_t i = tid; i < n; i += blockDim.x) od[pl[i]] = i;
    __syncthreads();
  }
  if (fg) {
    // Fusion groups: every member moves to the place of the group's best-ranked member and the
    // members stand there in layer order.  Places of different groups differ, so sorting by
    // (best place of my group, layer index) yields exactly that list.
    for (uint32_t i = tid; i < n; i += blockDim.x) {
      const uint32_t g = fg[i];
      uint32_t b = pl[i];
      if (g != kNoGroup)
        for (uint32_t j = 0; j < n; ++j)
          if (fg[j] == g) b = min(b, pl[j]);
      bs[i] = b;
    }
    __syncthreads();
    for (uint32_t i = tid; i < n; i += blockDim.x) {
      const uint32_t bi = bs[i];
      uint32_t rank = 0;
      for (uint32_t j = 0; j < n; ++j) {
        const uint32_t bj = bs[j];
        if (bj < bi || (bj == bi && j < i)) ++rank;
      }
      od[rank] = i;
    }
    __syncthreads();
  }
  // The FP32-kept prefix grows one whole fusion group at a time (a layer without a group is a group
  // of one): by count while it still fits, by rate while the rate still holds.  With K the MACs
  // kept so far, "quantized share >= rate" is (total - K) * 10000 >= rate * total, i.e.
  // K * 10000 <= total * (10000 - rate); 128-bit integers, exact.  Both tests only get harder as
  // the prefix grows, so the walk "stop at the first group that fails" ends at the LONGEST prefix
  // that ends on a group boundary and passes.
  if (staged) {
    // Every list position is tested by its own thread: MACs and groups gathered in list order, a
    // 128-bit prefix sum per position (n <= 512 additions each), then the largest passing cut.
    unsigned long long* p_lo = reinterpret_cast<unsigned long long*>(s_score);   // scores and severities
    unsigned long long* p_hi = reinterpret_cast<unsigned long long*>(s_sev);     // are no longer needed
    __shared__ uint32_t s_nk;
    if (tid == 0) s_nk = 0;
    for (uint32_t k = tid; k < n; k += blockDim.x) {
      const uint32_t l = od[k];
      s_mlist[k] = mc ? mc[l] : 1ull;
      s_best[k] = fg ? fg[l] : kNoGroup;
    }
    __syncthreads();
    const bool by_count = cfg.select_mode == QV2_BY_COUNT;
    if (!by_count) {
      for (uint32_t k = tid; k < n; k += blockDim.x) {
        unsigned __int128 acc = 0;
#pragma unroll 4
        for (uint32_t q = 0; q <= k; ++q) acc += s_mlist[q];
        p_lo[k] = (unsigned long long)acc; p_hi[k] = (unsigned long long)(acc >> 64);
      }
      __syncthreads();
    }
    const unsigned __int128 total = by_count ? 0 : (((unsigned __int128)p_hi[n - 1] << 64) | p_lo[n - 1]);
    const unsigned __int128 limit = total * (unsigned __int128)(10000u - cfg.rate_permyriad);
    for (uint32_t k = tid; k < n; k += blockDim.x) {
      const uint32_t e = k + 1, g = s_best[k];
      const bool boundary = e == n || g == kNoGroup || s_best[e] != g;
      bool pass;
      if (by_count) pass = e <= cfg.keep_count;
      else pass = ((((unsigned __int128)p_hi[k] << 64) | p_lo[k]) * 10000u) <= limit;
      if (boundary && pass) atomicMax(&s_nk, e);
    }
    __syncthreads();
    const uint32_t nk = s_nk;
    for (uint32_t k = tid; k < nk; k += blockDim.x) kp[od[k]] = 1;
    if (tid == 0) *n_keep = nk;
  } else if (tid == 0) {
    auto grp = [&](uint32_t l) { return fg ? fg[l] : kNoGroup; };
    auto mac = [&](uint32_t l) { return mc ? mc[l] : 1ull; };
    unsigned __int128 total = 0, kept = 0;
    if (cfg.select_mode != QV2_BY_COUNT)
      for (uint32_t i = 0; i < n; ++i) total += mac(i);
    const unsigned __int128 limit = total * (unsigned __int128)(10000u - cfg.rate_permyriad);
    uint32_t nk = 0, j = 0;
    while (j < n) {
      const uint32_t g = grp(od[j]);
      uint32_t e = j + 1;
      if (g != kNoGroup) while (e < n && grp(od[e]) == g) ++e;
      if (cfg.select_mode == QV2_BY_COUNT) {
        if (e <= cfg.keep_count) nk = e; else break;
      } else {
        unsigned __int128 m = 0;
        for (uint32_t k = j; k < e; ++k) m += mac(od[k]);
        if ((kept + m) * 10000u <= limit) { kept += m; nk = e; }
        else break;
      }
      j = e;
    }
    for (uint32_t k = 0; k < nk; ++k) kp[od[k]] = 1;
    *n_keep = nk;
  }
  if (staged) {                        // publish the list and the flags
    __syncthreads();
    for (uint32_t i = tid; i < n; i += blockDim.x) { order[i] = s_order[i]; keep[i] = s_keep[i]; }
  }
}

}  // namespace

cudaError_t launch_rank(const Launch& l, uint32_t n, const double* sqnr_w, const double* mse_w,
                        const double* sqnr_a, const double* mse_a, const uint64_t* macs,
                        const double* pos, const uint32_t* fuse_group, qv2_rank_cfg cfg, double* scratch,
                        uint32_t* order, uint8_t* keep, uint32_t* n_keep) {
  // scratch: kMaxRankLayers doubles each for score and severity, then two uint32 arrays
  uint32_t* place = reinterpret_cast<uint32_t*>(scratch + 2 * (size_t)kMaxRankLayers);
  return launch_kernel(l, rank_kernel, 1u, 256u, n, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, fuse_group, cfg, scratch,
                       scratch + kMaxRankLayers, place, place + kMaxRankLayers, order, keep, n_keep);
}

}  // namespace qv2

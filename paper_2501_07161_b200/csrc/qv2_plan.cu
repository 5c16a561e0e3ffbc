// Host planner: validates tensor descriptors and cuts a whole model's ragged layer list into the
// tile table that one kernel launch per phase walks (segmented multi-layer batching).
#include <new>

#include "qv2_common.cuh"

namespace qv2 {

static bool mul_overflows(uint64_t a, uint64_t b, uint64_t* out) {
  if (a != 0 && b > UINT64_MAX / a) return true;
  *out = a * b;
  return false;
}

static void cut_flat(uint32_t tensor, uint64_t begin, uint64_t count, uint64_t group,
                     std::vector<Tile>* tiles) {
  while (count > 0) {
    uint32_t c = count > kTileElems ? kTileElems : (uint32_t)count;
    Tile t;
    t.begin = begin; t.row0 = group; t.count = c; t.tensor = tensor; t.rows = 0; t.pack = 0;
    tiles->push_back(t);
    begin += c; count -= c;
  }
}

// Tables larger than this many tiles (4 GB of records; two trillion elements) are refused before
// any of them is generated.
constexpr uint64_t kMaxTiles = 1ull << 27;
constexpr uint64_t kMicroGroupMax = 2048;    // per-group histograms: groups this small are packed into micro units ...
constexpr uint64_t kMicroUnitElems = 8192;   // ... of about this many elements (the kernel needs the square to fit 32 bits)

static int build_plan_checked(const qv2_tensor_desc* descs, uint32_t n, const GridCaps& caps,
                              uint64_t chunk_bytes, uint32_t fold_mode, HostPlan* out) {
  if (!descs || !out) return QV2_ERR_NULL;
  if (n == 0 || n > 65535u) return QV2_ERR_SIZE;
  *out = HostPlan();
  out->tensors.reserve(n);
  std::vector<uint32_t> tile_cnt(n, 0), hist_cnt(n, 0);
  uint64_t groups = 0;
  bool any_group_pct = false;
  for (uint32_t t = 0; t < n; ++t) {
    const qv2_tensor_desc& d = descs[t];
    if (d.granularity > QV2_PER_CHANNEL || d.scheme > QV2_ASYM_U8_ZP || d.range > QV2_PERCENTILE_GROUP)
      return QV2_ERR_ARG;
    if (d.flags & ~(uint32_t)(QV2_PAIR_RAW | QV2_STORE_CODES | QV2_BITS_MASK | QV2_IN_MASK)) return QV2_ERR_ARG;
    const uint32_t dtype = (d.flags & QV2_IN_MASK) >> 16;
    if (dtype > kBF16) return QV2_ERR_ARG;
    const uint32_t bits = QV2_DESC_BITS(d.flags);
    if (bits < 2 || bits > 16) return QV2_ERR_ARG;
    if ((d.flags & QV2_STORE_CODES) && bits > 8) return QV2_ERR_UNSUPPORTED;   // codes are one byte
    if (d.range >= QV2_PERCENTILE && !(d.percentile >= 0.0 && d.percentile <= 1.0))
      return QV2_ERR_ARG;
    uint64_t rows, ne;
    if (mul_overflows(d.outer, d.channels, &rows) || rows > (1ull << 62)) return QV2_ERR_SIZE;
    if (mul_overflows(rows, d.inner, &ne) || ne > (1ull << 62)) return QV2_ERR_SIZE;
    if (d.channels >= (1ull << 32)) return QV2_ERR_SIZE;
    if (ne > 0 && !d.x) return QV2_ERR_NULL;
    const uintptr_t amask = dtype_size(dtype) - 1u;
    if (((uintptr_t)d.x & amask) || ((uintptr_t)d.y & amask)) return QV2_ERR_ALIGN;
    bool pair = d.y != nullptr;
    if ((d.flags & QV2_PAIR_RAW) && !pair) return QV2_ERR_ARG;

    TensorRec r = TensorRec();
    r.x = d.x; r.y = d.y;
    r.n_elems = ne; r.inner = d.inner;
    r.channels = (uint32_t)d.channels;
    r.per_channel = d.granularity == QV2_PER_CHANNEL;
    r.n_groups = r.per_channel ? (uint32_t)d.channels : 1u;
    if (groups + r.n_groups >= (1ull << 32)) return QV2_ERR_SIZE;
    r.group_base = (uint32_t)groups;
    groups += r.n_groups;
    r.asym = d.scheme;                  // 0 symmetric, 1 affine with real offset, 2 affine with zero point
    // one group: its histogram is the tensor's, so the per-group mode is the per-tensor one
    r.range_mode = (d.range == QV2_PERCENTILE_GROUP && !r.per_channel) ? (uint32_t)QV2_PERCENTILE : d.range;
    if (r.range_mode == QV2_PERCENTILE_GROUP) {
      if (out->ghist_owner.size() + r.n_groups >= (1ull << 32)) return QV2_ERR_SIZE;
      r.ghist_first = (uint32_t)out->ghist_owner.size();
      out->ghist_owner.insert(out->ghist_owner.end(), r.n_groups, t);
      any_group_pct = true;
    }
    r.pair_mode = !pair ? kSelf : ((d.flags & QV2_PAIR_RAW) ? kRaw : kRequant);
    r.percentile = d.percentile;
    r.bits = bits;
    r.dtype = dtype;
    if (dtype != kF32) out->any_16bit = true;

    const size_t first_tile = out->tiles.size(), first_hist = out->hist_tiles.size();
    {
      uint64_t need;
      if (ne == 0) need = 0;
      else if (!r.per_channel) need = (ne + kTileElems - 1) / kTileElems;
      else if (d.inner >= kRowTileMin) need = rows * ((d.inner + kTileElems - 1) / kTileElems);   // <= ne / 16384 + rows: no overflow
      else need = rows / (kTileElems / d.inner) + 1;             // kTileElems / inner >= 1 whole rows per tile
      if (need > kMaxTiles || out->tiles.size() + need > kMaxTiles) return QV2_ERR_SIZE;
      if (r.range_mode == QV2_PERCENTILE &&
          out->hist_tiles.size() + (ne + kTileElems - 1) / kTileElems > kMaxTiles) return QV2_ERR_SIZE;
    }
    if (r.range_mode == QV2_PERCENTILE) {
      out->any_percentile = true;
      r.hist_index = out->n_hist++;
    }
    if (ne > 0) {
      if (!r.per_channel) {
        cut_flat(t, 0, ne, 0, &out->tiles);
      } else if (d.inner >= kRowTileMin) {
        // (Cutting a row into equal tiles, or dealing its 8192-element rounds evenly so that no
        // tile is a sliver, was measured on 50176-element rows: the metrics kernel gains 3 %, the
        // range kernel loses as much, the pass stays within 0.6 % either way.)
        for (uint64_t row = 0; row < rows; ++row)
          cut_flat(t, row * d.inner, d.inner, row % d.channels, &out->tiles);
      } else {
        // whole rows, about kTileElems elements per tile.  (Tiles of 32 K and 64 K elements were
        // measured: the longer per-warp streams gain 1 % on VGG-16 shapes, the coarser balance loses
        // 5-10 % on ResNet-18 shapes.)
        const uint64_t per = kTileElems / d.inner;       // inner < kRowTileMin, so per >= 1
        for (uint64_t row = 0; row < rows; row += per) {
          uint64_t nr = rows - row < per ? rows - row : per;
          Tile tl;
          tl.begin = row * d.inner; tl.row0 = row; tl.count = (uint32_t)(nr * d.inner);
          tl.tensor = t; tl.rows = (uint32_t)nr; tl.pack = 0;
          out->tiles.push_back(tl);
        }
      }
      if (r.range_mode == QV2_PERCENTILE) cut_flat(t, 0, ne, 0, &out->hist_tiles);
      if (r.range_mode == QV2_PERCENTILE_GROUP) {
        // Group-major units for the per-group histograms: `rows` segments of `count` elements of
        // ONE group, segment k starting at begin + k * channels * inner (the same channel of the
        // next batch item).  A unit holds about kGroupUnitElems elements so that a CTA merges its
        // shared-memory histogram once per unit; rows longer than kGroupSegMax are cut.
        // Groups of at most kMicroGroupMax elements are packed instead: a unit is `pack`
        // consecutive channels (count = inner, rows = outer, begin at the first channel of batch
        // item 0), about kMicroUnitElems elements and at most one bin-scale table of channels.
        const uint64_t per = kGroupUnitElems / d.inner ? kGroupUnitElems / d.inner : 1;   // rows per unit
        const uint64_t group_elems = d.outer * d.inner;
        const bool micro = group_elems <= kMicroGroupMax;
        uint64_t pack = micro ? kMicroUnitElems / group_elems : 1;     // channels per micro unit
        if (pack > kBins) pack = kBins;
        const uint64_t per_group = d.inner > kGroupSegMax
            ? d.outer * ((d.inner + kGroupSegMax - 1) / kGroupSegMax) : (d.outer + per - 1) / per;
        uint64_t total;
        if (mul_overflows(per_group, d.channels, &total) || out->ghist_tiles.size() + total > (1ull << 26))
          return QV2_ERR_SIZE;
        for (uint64_t c = 0; c < d.channels; c += pack) {
          if (micro) {
            Tile u;
            u.begin = c * d.inner; u.row0 = c; u.count = (uint32_t)d.inner; u.tensor = t;
            u.rows = (uint32_t)d.outer; u.pack = (uint32_t)(d.channels - c < pack ? d.channels - c : pack);
            out->ghist_tiles.push_back(u);
          } else if (d.inner > kGroupSegMax) {
            for (uint64_t o = 0; o < d.outer; ++o)
              for (uint64_t off = 0; off < d.inner; off += kGroupSegMax) {
                Tile u;
                u.begin = (o * d.channels + c) * d.inner + off; u.row0 = c;
                u.count = (uint32_t)(d.inner - off < kGroupSegMax ? d.inner - off : kGroupSegMax);
                u.tensor = t; u.rows = 1; u.pack = 0;
                out->ghist_tiles.push_back(u);
              }
          } else {
            for (uint64_t o = 0; o < d.outer; o += per) {
              Tile u;
              u.begin = (o * d.channels + c) * d.inner; u.row0 = c; u.count = (uint32_t)d.inner;
              u.tensor = t; u.rows = (uint32_t)(d.outer - o < per ? d.outer - o : per); u.pack = 0;
              out->ghist_tiles.push_back(u);
            }
          }
        }
      }
    }
    if (out->tiles.size() >= (1ull << 31) || out->hist_tiles.size() >= (1ull << 31)) return QV2_ERR_SIZE;
    tile_cnt[t] = (uint32_t)(out->tiles.size() - first_tile);
    hist_cnt[t] = (uint32_t)(out->hist_tiles.size() - first_hist);
    out->tensors.push_back(r);
  }

  // Stages: runs of consecutive tensors.  A "resident" stage holds reference tensors of at most
  // chunk_bytes together; tensors larger than that gather in stages of their own, where a second
  // pass cannot hit L2 anyway.  Per-group histograms are walked by a separate table that is not
  // cut into stages, so a plan that has them keeps the single-stage schedule.
  {
    const bool chunked = chunk_bytes != 0 && !any_group_pct;
    Stage st = Stage();
    uint64_t held = 0;
    bool open = false, open_big = false;
    auto close = [&](uint32_t end) { st.tensor_end = end; out->stages.push_back(st); };
    for (uint32_t t = 0; t < n; ++t) {
      const TensorRec& r = out->tensors[t];
      const uint64_t bytes = r.n_elems * dtype_size(r.dtype);
      const bool big = chunked && bytes > chunk_bytes;
      const bool fits = open && (!chunked || (big && open_big) || (!big && !open_big && held + bytes <= chunk_bytes));
      if (open && !fits) { close(t); open = false; }
      if (!open) { st = Stage(); st.tensor_begin = t; st.l2_resident = chunked && !big; held = 0; open = true; open_big = big; }
      held += bytes;
    }
    close(n);
  }

  // Slots written with plain stores instead of atomics.  In every persistent kernel CTA b walks
  // tiles b, b+grid, ... of its stage's slice; a tensor whose tiles are [first, first+count) is
  // therefore touched by min(grid, count) CTAs.  The metrics kernel gives each of those CTAs one
  // partial-sum slot; the range kernel gives each of them one {min,max} slot for per-tensor
  // tensors (a single group shared by thousands of tiles; per-channel groups are merged with
  // atomics).
  uint64_t slots = 0, rslots = 0, tile_at = 0, hist_at = 0;
  for (Stage& st : out->stages) {
    st.tile_begin = (uint32_t)tile_at; st.hist_begin = (uint32_t)hist_at;
    uint64_t nt = 0, nh = 0;
    for (uint32_t t = st.tensor_begin; t < st.tensor_end; ++t) { nt += tile_cnt[t]; nh += hist_cnt[t]; }
    st.tile_end = (uint32_t)(tile_at + nt); st.hist_end = (uint32_t)(hist_at + nh);
    auto grid_of = [](uint32_t cap, uint64_t tiles) -> uint32_t {
      uint64_t g = cap < 1 ? 1 : cap;
      if (g > tiles) g = tiles;
      return g < 1 ? 1u : (uint32_t)g;
    };
    uint64_t swept = 0;                    // bytes one metrics launch of the stage reads
    for (uint32_t t = st.tensor_begin; t < st.tensor_end; ++t) {
      const TensorRec& r = out->tensors[t];
      swept += r.n_elems * dtype_size(r.dtype) * (r.y ? 2u : 1u);
    }
    st.fused_fold = fold_mode == QV2_FOLD_AUTO ? swept <= kFusedFoldMaxBytes : fold_mode == QV2_FOLD_FUSED;
    st.range_grid = grid_of(st.fused_fold ? caps.range_fused : caps.range, nt);
    st.metrics_grid = grid_of(st.fused_fold ? caps.metrics_fused : caps.metrics, nt);
    st.hist_grid = grid_of(st.fused_fold ? caps.hist_fused : caps.hist, nh);
    uint64_t rel = 0, hrel = 0;
    for (uint32_t t = st.tensor_begin; t < st.tensor_end; ++t) {
      TensorRec& r = out->tensors[t];
      r.tile_first = (uint32_t)rel; r.hist_tile_first = (uint32_t)hrel;
      rel += tile_cnt[t]; hrel += hist_cnt[t];
      r.metrics_ctas = tile_cnt[t] < st.metrics_grid ? tile_cnt[t] : st.metrics_grid;
      r.range_ctas = tile_cnt[t] < st.range_grid ? tile_cnt[t] : st.range_grid;
      r.hist_ctas = hist_cnt[t] < st.hist_grid ? hist_cnt[t] : st.hist_grid;
      if (slots + r.metrics_ctas >= (1ull << 32)) return QV2_ERR_SIZE;
      r.slot_first = (uint32_t)slots;
      slots += r.metrics_ctas;
      if (!r.per_channel) {
        if (rslots + r.range_ctas >= (1ull << 32)) return QV2_ERR_SIZE;
        r.rslot_first = (uint32_t)rslots;
        rslots += r.range_ctas;
      }
      if (tile_cnt[t] == 0) st.any_empty = true;
      if (r.range_mode == QV2_PERCENTILE) st.any_percentile = true;
    }
    tile_at += nt; hist_at += nh;
  }
  out->total_rslots = (uint32_t)rslots;
  out->total_groups = groups;
  out->total_slots = (uint32_t)slots;
  return QV2_OK;
}

int build_plan(const qv2_tensor_desc* descs, uint32_t n, const GridCaps& caps, uint64_t chunk_bytes,
               uint32_t fold_mode, HostPlan* out) {
  try {
    return build_plan_checked(descs, n, caps, chunk_bytes, fold_mode, out);
  } catch (const std::bad_alloc&) {          // nothing may unwind through the C ABI
    return QV2_ERR_NOMEM;
  }
}

}  // namespace qv2

extern "C" uint64_t qv2_group_count(const qv2_tensor_desc* descs, uint32_t n) {
  uint64_t g = 0;
  if (!descs) return 0;
  for (uint32_t t = 0; t < n; ++t)
    g += descs[t].granularity == QV2_PER_CHANNEL ? descs[t].channels : 1;
  return g;
}

extern "C" uint64_t qv2_group_hist_count(const qv2_tensor_desc* descs, uint32_t n) {
  uint64_t g = 0;
  if (!descs) return 0;
  for (uint32_t t = 0; t < n; ++t)
    if (descs[t].range == QV2_PERCENTILE_GROUP && descs[t].granularity == QV2_PER_CHANNEL) g += descs[t].channels;
  return g;
}

extern "C" int64_t qv2_debug_plan_tiles(const qv2_tensor_desc* descs, uint32_t n, uint64_t* out,
                                        uint64_t max_tiles) {
  qv2::HostPlan plan;
  int st = qv2::build_plan(descs, n, qv2::GridCaps(), 0, QV2_FOLD_AUTO, &plan);
  if (st != QV2_OK) return st;
  uint64_t w = 0;
  for (const qv2::Tile& t : plan.tiles) {
    if (w >= max_tiles || !out) break;
    out[4 * w + 0] = t.tensor; out[4 * w + 1] = t.begin; out[4 * w + 2] = t.count;
    out[4 * w + 3] = t.rows ? 1 : 0;
    ++w;
  }
  return (int64_t)plan.tiles.size();
}

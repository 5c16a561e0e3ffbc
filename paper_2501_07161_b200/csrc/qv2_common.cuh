// Shared declarations of the qv2 CUDA library: device-side records, the tile decomposition and
// the launch wrappers each kernel file exports to the C-ABI layer.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/qv2.h"

namespace qv2 {

constexpr int kThreads = 256;            // threads per CTA in the streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kTileElems = 16384;   // elements per tile (64 KiB of fp32)
constexpr uint64_t kRowTileMin = 4096;   // rows at least this long are cut into one-group tiles
constexpr uint64_t kShortRow = 128;      // rows shorter than this are walked element-parallel, longer ones one warp per row
constexpr uint64_t kGroupUnitElems = 131072;   // elements per unit of the per-group histogram pass
constexpr uint64_t kGroupSegMax = 1ull << 22;   // longest contiguous segment of such a unit
constexpr int kBins = QV2_HIST_BINS;
constexpr uint32_t kMaxRankLayers = 8192;

enum PairMode : uint32_t { kSelf = 0, kRequant = 1, kRaw = 2 };
enum DType : uint32_t { kF32 = 0, kF16 = 1, kBF16 = 2 };
inline uint32_t dtype_size(uint32_t dtype) { return dtype == kF32 ? 4u : 2u; }

// One tensor, as the kernels see it.
struct TensorRec {
  const float* x;
  const float* y;
  uint8_t* codes;            // nullable
  uint64_t n_elems;
  uint64_t inner;
  uint32_t channels;
  uint32_t group_base;       // index of this tensor's group 0 in the per-group arrays
  uint32_t n_groups;
  uint32_t per_channel;
  uint32_t asym;             // 0: symmetric, 1: affine with real offset, 2: affine with integer zero point
  uint32_t range_mode;       // QV2_ABSMAX | QV2_MINMAX | QV2_PERCENTILE | QV2_PERCENTILE_GROUP (per-channel only)
  uint32_t pair_mode;        // PairMode
  uint32_t slot_first;       // first partial-sum slot of this tensor
  uint32_t slot_count;       // kWarps slots for every CTA of the metrics grid that owns a tile of it
  uint32_t tile_first;       // index of this tensor's first tile in the tile table
  uint32_t rslot_first;      // per-tensor tensors: first {min,max} key slot written by the range kernel,
  uint32_t rslot_count;      //   one per CTA of the range grid that owns a tile of the tensor
  uint32_t bits;             // code width, 2..16 (8 unless the descriptor asks otherwise)
  uint32_t dtype;            // element type of x and y: 0 binary32, 1 binary16, 2 bfloat16
  uint32_t ghist_first;      // QV2_PERCENTILE_GROUP: index of group 0's histogram among the per-group histograms
  double percentile;
};

// A contiguous run of elements of one tensor handled by one CTA at a time.
//  rows == 0: every element belongs to quantization group `row0` (0 for per-tensor tensors).
//  rows  > 0: `rows` whole rows of `inner` elements starting at row `row0`; the group of row r
//             is r % channels.
struct Tile {
  uint64_t begin;
  uint64_t row0;
  uint32_t count;
  uint32_t tensor;
  uint32_t rows;
  uint32_t reserved;
};
static_assert(sizeof(Tile) == 32, "Tile is read as two 16-byte words");

struct HostPlan {
  std::vector<TensorRec> tensors;
  std::vector<Tile> tiles;        // every tensor, in tensor order
  std::vector<Tile> hist_tiles;   // flat tiles of the tensors that need a histogram
  std::vector<Tile> ghist_tiles;  // group-major units of the tensors that need per-group histograms (see build_plan)
  std::vector<uint32_t> ghist_owner;   // per-group histogram -> tensor index
  uint64_t total_groups = 0;
  uint32_t total_slots = 0;
  uint32_t metrics_grid = 1;      // CTAs of the metrics launch; the slot layout depends on it
  uint32_t total_rslots = 0;
  uint32_t range_grid = 1;        // CTAs of the range launch; the range-slot layout depends on it
  bool any_percentile = false;
  bool any_16bit = false;         // some tensor is stored in binary16 / bfloat16
};

// Validates the descriptors and cuts them into tiles.  `codes` may be NULL.  `metrics_cap` and
// `range_cap` are the largest useful grids of those kernels (resident CTAs per SM x SMs).
// Returns a QV2 status.
int build_plan(const qv2_tensor_desc* descs, uint32_t n, void* const* codes, uint32_t metrics_cap,
               uint32_t range_cap, HostPlan* out);

// ------------------------------------------------------------------------------------------------
// Launch wrappers (defined next to their kernels).  All enqueue on `stream` and return the
// cudaError_t of the launch.
struct Launch {
  cudaStream_t stream;
  int sm_count;
};

cudaError_t launch_range(const Launch& l, uint32_t grid, bool any16, const TensorRec* tensors, const Tile* tiles,
                         uint32_t n_tiles, uint32_t* kmin, uint32_t* kmax, uint2* rslots,
                         unsigned long long* nonfinite);
cudaError_t launch_calib_init(const Launch& l, uint32_t* kmin, uint32_t* kmax, size_t groups,
                              unsigned long long* nonfinite, size_t n_tensors, unsigned long long* hist,
                              size_t hist_cells);
uint32_t range_grid_cap(int sm_count);     // resident CTAs per SM x SMs for the range kernel
cudaError_t launch_range_finalize(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                  const uint2* rslots, float* gmin, float* gmax, float* gabsmax,
                                  float* step, float* inv, float* offset, float* tensor_absmax, float* clip);
cudaError_t launch_hist(const Launch& l, bool any16, const TensorRec* tensors, const Tile* tiles,
                        uint32_t n_tiles, const float* tensor_absmax,
                        const unsigned long long* nonfinite, unsigned long long* hist);
cudaError_t launch_clip_finalize(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                 const unsigned long long* hist, const float* tensor_absmax,
                                 const float* gmin, const float* gmax, const float* gabsmax,
                                 float* clip, float* step, float* inv, float* offset);
cudaError_t launch_group_hist(const Launch& l, bool any16, const TensorRec* tensors, const Tile* tiles,
                              uint32_t n_tiles, const float* gabsmax, const unsigned long long* nonfinite,
                              unsigned long long* ghist);
cudaError_t launch_group_clip_finalize(const Launch& l, const TensorRec* tensors, const uint32_t* owner,
                                       uint32_t n_hists, const unsigned long long* ghist,
                                       const float* gmin, const float* gmax, const float* gabsmax,
                                       float* group_clip, float* step, float* inv, float* offset);
cudaError_t launch_fill_group_clip(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                   const float* clip, float* group_clip);
cudaError_t launch_metrics(const Launch& l, uint32_t grid, bool any16, const TensorRec* tensors,
                           const Tile* tiles, uint32_t n_tiles, const float* step, const float* inv,
                           const float* offset, double2* partials, double* partials_xe);
uint32_t metrics_grid_cap(int sm_count);   // resident CTAs per SM x SMs for the metrics kernel
cudaError_t launch_metrics_finalize(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                    const double2* partials, const double* partials_xe, double* sse,
                                    double* sig, double* mse, double* sqnr_db, double* cosine);
cudaError_t launch_kl(const Launch& l, const TensorRec* tensors, uint32_t n_tensors, const Tile* tiles,
                      uint32_t n_tiles, const float* step, const float* inv, const float* offset,
                      const float* gabsmax, float* tensor_absmax, unsigned long long* hists, double* kl);
cudaError_t launch_fold(const Launch& l, const float* w, const float* bias, const float* gamma,
                        const float* beta, const float* mean, const float* var, uint64_t channels,
                        uint64_t inner, float* w_out, float* bias_out);
cudaError_t launch_rank(const Launch& l, uint32_t n, const double* sqnr_w, const double* mse_w,
                        const double* sqnr_a, const double* mse_a, const uint64_t* macs,
                        const double* pos, const uint32_t* fuse_group, qv2_rank_cfg cfg, double* scratch,
                        uint32_t* order, uint8_t* keep, uint32_t* n_keep);
constexpr size_t kRankScratchDoubles = 3 * (size_t)kMaxRankLayers;   // see launch_rank

}  // namespace qv2

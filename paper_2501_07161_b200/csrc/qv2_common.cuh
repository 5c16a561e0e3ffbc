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
constexpr uint64_t kRowTileMin = 16384;  // rows at least this long are cut into one-group tiles walked by the whole CTA;
                                         // shorter rows come as tiles of whole rows (about kTileElems elements) and are
                                         // walked by the row walkers of each kernel, which keep eight streams per CTA going
                                         // whatever the row length (a 4608-element row walked by the whole CTA is a single
                                         // round of loads followed by a drain)
constexpr uint64_t kGroupUnitElems = 131072;   // elements per unit of the per-group histogram pass
constexpr uint64_t kGroupSegMax = 1ull << 22;   // longest contiguous segment of such a unit
constexpr int kBins = QV2_HIST_BINS;
constexpr uint32_t kMaxRankLayers = 8192;

enum PairMode : uint32_t { kSelf = 0, kRequant = 1, kRaw = 2 };
enum DType : uint32_t { kF32 = 0, kF16 = 1, kBF16 = 2 };
inline uint32_t dtype_size(uint32_t dtype) { return dtype == kF32 ? 4u : 2u; }

// One tensor, as the kernels see it.
//
// A pass is cut into stages (see HostPlan); each phase of a stage is one launch that walks the
// stage's slice of the tile table.  `tile_first` / `hist_tile_first` are relative to that slice,
// and the *_ctas fields count the CTAs of that launch that own at least one tile of the tensor:
// CTA b of a grid of g walks tiles b, b+g, ..., so a tensor whose tiles are [first, first+count)
// is touched by min(g, count) CTAs, numbered rank = (b - first) mod g.  The CTA that is last to
// finish its share of a tensor (an atomic ticket, never a wait) folds the tensor's partial
// results; the slot fields say where those partial results live.
struct TensorRec {
  const float* x;
  const float* y;
  uint64_t n_elems;
  uint64_t inner;
  uint32_t channels;
  uint32_t group_base;       // index of this tensor's group 0 in the per-group arrays
  uint32_t n_groups;
  uint32_t per_channel;
  uint32_t asym;             // 0: symmetric, 1: affine with real offset, 2: affine with integer zero point
  uint32_t range_mode;       // QV2_ABSMAX | QV2_MINMAX | QV2_PERCENTILE | QV2_PERCENTILE_GROUP (per-channel only)
  uint32_t pair_mode;        // PairMode
  uint32_t tile_first;       // index of this tensor's first tile in its stage's slice of the tile table
  uint32_t hist_tile_first;  // the same in the slice of the histogram tile table (percentile tensors)
  uint32_t slot_first;       // first partial-sum slot of this tensor, one per CTA of the metrics launch
  uint32_t metrics_ctas;     //   that owns a tile of it
  uint32_t rslot_first;      // per-tensor tensors: first {min,max} key slot written by the range kernel
  uint32_t range_ctas;       // CTAs of the range launch that own a tile of the tensor
  uint32_t hist_ctas;        // CTAs of the histogram launch that own a tile of the tensor
  uint32_t hist_index;       // percentile tensors: index of the tensor's accumulation histogram in scratch
  uint32_t bits;             // code width, 2..16 (8 unless the descriptor asks otherwise)
  uint32_t dtype;            // element type of x and y: 0 binary32, 1 binary16, 2 bfloat16
  uint32_t ghist_first;      // QV2_PERCENTILE_GROUP: index of group 0's histogram among the per-group histograms
  uint32_t reserved[2];
  double percentile;
};

// A contiguous run of elements of one tensor handled by one CTA at a time.
//  rows == 0: every element belongs to quantization group `row0` (0 for per-tensor tensors).
//  rows  > 0: `rows` whole rows of `inner` elements starting at row `row0`; the group of row r
//             is r % channels.
// In the unit table of the per-group histograms a record means something else: `rows` segments
// of `count` elements of group `row0`, segment k at begin + k * channels * inner; and when
// `pack` > 0, `pack` consecutive groups row0, row0 + 1, ... taken together (count = inner,
// rows = outer).  `pack` is 0 in the tile tables.
struct Tile {
  uint64_t begin;
  uint64_t row0;
  uint32_t count;
  uint32_t tensor;
  uint32_t rows;
  uint32_t pack;
};
static_assert(sizeof(Tile) == 32, "Tile is read as two 16-byte words");

// A run of consecutive tensors whose phases are launched together.  The phase-major schedule has
// one stage (every tensor); the L2-chunked schedule cuts the model into stages whose reference
// tensors fit in L2 together, and runs range -> histogram -> metrics stage by stage, so that the
// second and third pass over a tensor are served from L2.
struct Stage {
  uint32_t tensor_begin, tensor_end;
  uint32_t tile_begin, tile_end;          // slice of HostPlan::tiles
  uint32_t hist_begin, hist_end;          // slice of HostPlan::hist_tiles
  uint32_t range_grid, hist_grid, metrics_grid;
  bool any_empty;                         // some tensor of the stage has no element (no CTA owns it)
  bool any_percentile;                    // some tensor of the stage is clipped at its percentile
  bool l2_resident;                       // the stage's reference tensors fit the chunk budget
  bool fused_fold;                        // small stage: the streaming kernels fold each tensor themselves (the CTA
                                          // that finishes it last); large stage: lean streaming kernels, each
                                          // followed by a small fold kernel with one CTA per tensor
};
// QV2_FOLD_AUTO takes the fused fold for stages that sweep at most this many bytes per phase.
// Zero: never.  Measured on a B200, the fused kernels lose more at their per-tensor barriers (every
// warp of a CTA drains its loads before the CTA publishes, 560 against 86 barrier-stall samples in
// the range kernel on ResNet-18 shapes) than the saved launches return, even for a 62 MB model
// replayed from a CUDA graph (30.8 against 28.7 us); the mode stays available on request.
constexpr uint64_t kFusedFoldMaxBytes = 0;

// Largest useful grid of each persistent kernel on the context's device (resident CTAs per SM x SMs).
// The streaming kernels come in two builds with different register counts (fold inside or not).
struct GridCaps {
  uint32_t range = 1, hist = 1, metrics = 1, ghist = 1, kl = 1;
  uint32_t range_fused = 1, hist_fused = 1, metrics_fused = 1;
};

struct HostPlan {
  std::vector<TensorRec> tensors;
  std::vector<Tile> tiles;        // every tensor, in tensor order
  std::vector<Tile> hist_tiles;   // flat tiles of the tensors that need a histogram
  std::vector<Tile> ghist_tiles;  // group-major units of the tensors that need per-group histograms (see build_plan)
  std::vector<uint32_t> ghist_owner;   // per-group histogram -> tensor index
  std::vector<Stage> stages;
  uint64_t total_groups = 0;
  uint32_t total_slots = 0;
  uint32_t total_rslots = 0;
  uint32_t n_hist = 0;            // tensors clipped at a per-tensor percentile (accumulation histograms in scratch)
  bool any_percentile = false;
  bool any_16bit = false;         // some tensor is stored in binary16 / bfloat16
};

// Validates the descriptors and cuts them into tiles and stages.  chunk_bytes == 0 gives the
// phase-major schedule (one stage); otherwise consecutive tensors are grouped into stages whose
// reference tensors hold at most chunk_bytes (a larger tensor gets a stage of its own kind).
// Returns a QV2 status.
// fold_mode: QV2_FOLD_AUTO decides per stage by its size, QV2_FOLD_FUSED / QV2_FOLD_SEPARATE force it.
int build_plan(const qv2_tensor_desc* descs, uint32_t n, const GridCaps& caps, uint64_t chunk_bytes,
               uint32_t fold_mode, HostPlan* out);

// ------------------------------------------------------------------------------------------------
// Launch wrappers (defined next to their kernels).  All enqueue on `stream` and return the
// cudaError_t of the launch.
struct Launch {
  cudaStream_t stream;
  int sm_count;
  bool pdl;            // launch as a programmatic dependent of the previous kernel in the stream
};

// Launches `kernel`; with l.pdl the launch may begin while the previous kernel of the stream is
// still draining (programmatic dependent launch).  Every kernel launched this way calls
// dependency_wait() before it reads or writes anything a previous kernel may touch.
template <class... KArgs, class... Args>
inline cudaError_t launch_kernel(const Launch& l, void (*kernel)(KArgs...), uint32_t grid, uint32_t block,
                                 Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = 0; cfg.stream = l.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = l.pdl ? 1u : 0u;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(static_cast<Args&&>(args))...);
}

// Scratch and outputs of the calibration phases.  Accumulators (keys, counters, histograms,
// tickets) are zero between passes: the CTA that folds a tensor clears what it consumed.
struct CalibArgs {
  const TensorRec* tensors;
  uint32_t* kmin; uint32_t* kmax;            // scratch: order-preserving keys per group, 0 = nothing seen
  uint2* rslots;                             // scratch: {min,max} key pair per CTA of a per-tensor tensor
  unsigned long long* nf_acc;                // scratch: non-finite counter per tensor
  unsigned long long* hist_acc;              // scratch: 2048 bins per percentile tensor
  uint32_t* tickets;                         // scratch: one per tensor, range phase
  uint32_t* hist_tickets;                    // scratch: one per tensor, histogram phase
  float* tensor_absmax;                      // scratch: per tensor
  float *gmin, *gmax, *gabsmax, *step, *inv, *offset;   // outputs, per group
  float* clip;                               // output, per tensor
  unsigned long long* nonfinite;             // output, per tensor
  unsigned long long* hist;                  // output, 2048 per tensor, nullable
};

cudaError_t launch_range(const Launch& l, const Stage& st, bool any16, const Tile* tiles, const CalibArgs& a);
cudaError_t launch_hist(const Launch& l, const Stage& st, bool any16, const Tile* hist_tiles, const CalibArgs& a);
uint32_t range_grid_cap(int sm_count, bool fused);     // resident CTAs per SM x SMs
uint32_t hist_grid_cap(int sm_count, bool fused);
uint32_t group_hist_grid_cap(int sm_count);
uint32_t metrics_grid_cap(int sm_count, bool fused);
uint32_t kl_grid_cap(int sm_count);

cudaError_t launch_group_hist(const Launch& l, uint32_t grid_cap, bool any16, const TensorRec* tensors,
                              const Tile* tiles, uint32_t n_tiles, const float* gabsmax,
                              const unsigned long long* nonfinite, unsigned long long* ghist);
cudaError_t launch_group_clip_finalize(const Launch& l, const TensorRec* tensors, const uint32_t* owner,
                                       uint32_t n_hists, const unsigned long long* ghist,
                                       const unsigned long long* nonfinite,
                                       const float* gmin, const float* gmax, const float* gabsmax,
                                       float* group_clip, float* step, float* inv, float* offset);
cudaError_t launch_fill_group_clip(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                   const float* clip, float* group_clip);

struct MetricsArgs {
  const TensorRec* tensors;
  const float *step, *inv, *offset;          // per group
  uint8_t* const* codes;                     // device table of per-tensor code buffers, nullable
  double2* partials;                         // scratch: {sum e^2, sum x^2} per CTA and tensor
  double* partials_xe;                       // scratch: sum x*e, cosine only (nullable)
  uint32_t* tickets;                         // scratch: one per tensor, metrics phase
  double *sse, *sig, *mse, *sqnr_db, *cosine;   // outputs per tensor (cosine nullable)
};
cudaError_t launch_metrics(const Launch& l, const Stage& st, bool any16, const Tile* tiles, const MetricsArgs& a);

cudaError_t launch_kl(const Launch& l, uint32_t grid_cap, const TensorRec* tensors, uint32_t n_tensors,
                      const Tile* tiles, uint32_t n_tiles, const float* step, const float* inv,
                      const float* offset, const float* gabsmax, float* tensor_absmax,
                      unsigned long long* hists, double* kl);
cudaError_t launch_fold(const Launch& l, const float* w, const float* bias, const float* gamma,
                        const float* beta, const float* mean, const float* var, uint64_t channels,
                        uint64_t inner, float* w_out, float* bias_out);
cudaError_t launch_rank(const Launch& l, uint32_t n, const double* sqnr_w, const double* mse_w,
                        const double* sqnr_a, const double* mse_a, const uint64_t* macs,
                        const double* pos, const uint32_t* fuse_group, qv2_rank_cfg cfg, double* scratch,
                        uint32_t* order, uint8_t* keep, uint32_t* n_keep);
constexpr size_t kRankScratchDoubles = 3 * (size_t)kMaxRankLayers;   // see launch_rank

}  // namespace qv2

// Fused fake-quantize / dequantize / error reduction -- the memory-bound core of the sweep
// (CalculateSQNR and CalculateMSE of Algorithm 2; quantizer Eq. 1 / Eq. 5, dequantizer Eq. 3,
// SQNR Eq. 6, MSE Eq. 7).
//
// One persistent launch walks the tile table of a whole model; CTA b takes tiles b, b+grid, ...
// Every lane reduces its share of a tile in binary32 (independent accumulators per vector lane),
// adds the tile's two sums to binary64 running sums that it keeps while the CTA stays on the same
// tensor, and when the tensor changes the CTA folds its lanes and warps in a fixed order and writes
// one {sum e^2, sum x^2} pair to its own slot.  The CTA that finishes a tensor last (an atomic
// ticket) adds the tensor's slots in a fixed order in binary64 and writes the metrics.  There are
// no floating-point atomics and no inter-CTA waits: for a given grid size the result is
// bit-identical from run to run.
#include <mutex>
#include <type_traits>

#include "qv2_device.cuh"

namespace qv2 {

namespace {

struct QP {
  float step, inv, off, qmin, qmax;
  float bias;   // added to the rounded value to form the stored code (the zero point, else 0)
};

// Per-lane accumulators of one tile.  AccCos also carries sum x*e, from which the cosine
// similarity of Eq. 8 follows without a second pass: A.B = sig - xe, |B|^2 = sig - 2 xe + sse.
struct Acc {
  static constexpr bool kWantsB = false;     // needs (x, e) only
  float sse, sig;
  __device__ __forceinline__ void clear() { sse = 0.0f; sig = 0.0f; }
  __device__ __forceinline__ void add(float x, float e) {
    sse = __fmaf_rn(e, e, sse);
    sig = __fmaf_rn(x, x, sig);
  }
  // fresh(): an accumulator that starts from nothing; fold(): four into one, fixed association;
  // merge(): add another accumulator's sums
  __device__ __forceinline__ Acc fresh() const { Acc r; r.clear(); return r; }
  __device__ __forceinline__ static Acc fold(const Acc* a) {
    Acc r;
    r.sse = __fadd_rn(__fadd_rn(a[0].sse, a[1].sse), __fadd_rn(a[2].sse, a[3].sse));
    r.sig = __fadd_rn(__fadd_rn(a[0].sig, a[1].sig), __fadd_rn(a[2].sig, a[3].sig));
    return r;
  }
  __device__ __forceinline__ void merge(const Acc& r) { sse = __fadd_rn(sse, r.sse); sig = __fadd_rn(sig, r.sig); }
};
struct AccCos {
  static constexpr bool kWantsB = false;
  float sse, sig, xe;
  __device__ __forceinline__ void clear() { sse = 0.0f; sig = 0.0f; xe = 0.0f; }
  __device__ __forceinline__ void add(float x, float e) {
    sse = __fmaf_rn(e, e, sse);
    sig = __fmaf_rn(x, x, sig);
    xe = __fmaf_rn(x, e, xe);
  }
  __device__ __forceinline__ AccCos fresh() const { AccCos r; r.clear(); return r; }
  __device__ __forceinline__ static AccCos fold(const AccCos* a) {
    AccCos r;
    r.sse = __fadd_rn(__fadd_rn(a[0].sse, a[1].sse), __fadd_rn(a[2].sse, a[3].sse));
    r.sig = __fadd_rn(__fadd_rn(a[0].sig, a[1].sig), __fadd_rn(a[2].sig, a[3].sig));
    r.xe = __fadd_rn(__fadd_rn(a[0].xe, a[1].xe), __fadd_rn(a[2].xe, a[3].xe));
    return r;
  }
  __device__ __forceinline__ void merge(const AccCos& r) {
    sse = __fadd_rn(sse, r.sse); sig = __fadd_rn(sig, r.sig); xe = __fadd_rn(xe, r.xe);
  }
};

// One element.  MODE: kSelf quantizes x, kRequant quantizes y on x's grid, kRaw compares x and y.
//  t  = fl(fl(v - off) * inv)                      (v - 0 == v exactly, so OFF=false skips it)
//  q  = rne(clamp(t)) == clamp(rne(t)) since the bounds are integers; the add/subtract of
//       1.5*2^23 rounds to nearest-even for |t| <= 2^22
//  e  = (x - off) - q*step, with x - off split exactly into (s, err) by TwoSum when off != 0 and
//       the product folded into one fused multiply-add, so e carries a single rounding error.
template <uint32_t MODE, bool OFF, bool CODES, class ACC>
__device__ __forceinline__ void metric_elem(float x, float y, const QP& p, ACC& a, uint8_t* code) {
  float e;
  if (MODE == kRaw) {
    e = __fsub_rn(x, y);
  } else {
    const float v = (MODE == kRequant) ? y : x;
    const float u = OFF ? __fsub_rn(v, p.off) : v;
    const float t = __fmul_rn(u, p.inv);
    const float tc = fminf(fmaxf(t, p.qmin), p.qmax);       // NaN -> qmin
    const float q = __fsub_rn(__fadd_rn(tc, 12582912.0f), 12582912.0f);
    if (OFF) {
      const float b = -p.off;
      const float s = __fadd_rn(x, b);
      const float bb = __fsub_rn(s, x);
      const float err = __fadd_rn(__fsub_rn(x, __fsub_rn(s, bb)), __fsub_rn(b, bb));
      e = __fadd_rn(__fmaf_rn(-q, p.step, s), err);
    } else {
      e = __fmaf_rn(-q, p.step, x);
    }
    if (CODES) *code = (uint8_t)(int)(q + p.bias);
    if constexpr (ACC::kWantsB) {
      // the compared value itself, in binary32 with fixed rounding points: fl(fl(q*step) + off)
      const float b = OFF ? __fadd_rn(__fmul_rn(q, p.step), p.off) : __fmul_rn(q, p.step);
      a.add_b(x, b);
      return;
    }
  }
  if constexpr (ACC::kWantsB) a.add_b(x, y);
  else a.add(x, e);
}

template <uint32_t MODE, bool OFF, bool CODES, class ACC>
__device__ __forceinline__ void metric_vec(const float4& x, const float4& y, const QP& p, ACC* a,
                                           uint8_t* code) {
  metric_elem<MODE, OFF, CODES>(x.x, y.x, p, a[0], code);
  metric_elem<MODE, OFF, CODES>(x.y, y.y, p, a[1], code + 1);
  metric_elem<MODE, OFF, CODES>(x.z, y.z, p, a[2], code + 2);
  metric_elem<MODE, OFF, CODES>(x.w, y.w, p, a[3], code + 3);
}

// This thread's share of a flat one-group run walked by STRIDE threads (the whole CTA, or one
// warp with tid = lane).  T is the element type of x and y in memory; `vec_y` says y has the same
// phase as x inside its group of four elements.
template <uint32_t MODE, bool OFF, bool CODES, uint32_t STRIDE = kThreads, class ACC, class T>
__device__ __forceinline__ void metric_flat(const T* __restrict__ x, const T* __restrict__ y,
                                            uint8_t* codes, uint32_t count, const QP& p, ACC* a,
                                            uint32_t tid = threadIdx.x) {
  constexpr bool PAIR = MODE != kSelf;
  const FlatSplit s = split_flat(x, count);
  const T* xb = x + s.head;
  const T* yb = PAIR ? y + s.head : nullptr;
  uint8_t* cb = CODES ? codes + s.head : nullptr;
  const bool vec_y = !PAIR || ((((uintptr_t)yb) & (4u * sizeof(T) - 1u)) == 0);
  uint32_t j = tid;
  if (vec_y) {
    constexpr uint32_t U = (PAIR ? 4 : 8) * (sizeof(T) == 2 ? 2 : 1);   // 16-bit elements: the same bytes in flight
    // Full rounds while EVERY thread of the walk still has U groups (the same trip count for all of
    // them: a warp never runs a round for a few of its lanes), then one predicated round with all
    // loads in flight for what is left.
    const uint32_t n_full = s.nvec / (U * STRIDE) * (U * STRIDE);
    for (; j < n_full; j += U * STRIDE) {
      float4 vx[U], vy[U];
#pragma unroll
      for (uint32_t u = 0; u < U; ++u) {
        vx[u] = ld_vec_at(xb, j + u * STRIDE);
        if (PAIR) vy[u] = ld_vec_at(yb, j + u * STRIDE); else vy[u] = vx[u];
      }
#pragma unroll
      for (uint32_t u = 0; u < U; ++u)
        metric_vec<MODE, OFF, CODES>(vx[u], vy[u], p, a, CODES ? cb + 4u * (j + u * STRIDE) : nullptr);
    }
    if (n_full < s.nvec) {          // fewer than U * STRIDE groups are left for the walk
      float4 vx[U], vy[U];
#pragma unroll
      for (uint32_t u = 0; u < U; ++u) {
        const uint32_t k = min(j + u * STRIDE, s.nvec - 1u);       // in bounds, maybe unused
        vx[u] = ld_vec_at(xb, k);
        if (PAIR) vy[u] = ld_vec_at(yb, k); else vy[u] = vx[u];
      }
#pragma unroll
      for (uint32_t u = 0; u < U; ++u)
        if (j + u * STRIDE < s.nvec)
          metric_vec<MODE, OFF, CODES>(vx[u], vy[u], p, a, CODES ? cb + 4u * (j + u * STRIDE) : nullptr);
    }
  } else {
    // x and y sit at different offsets inside their groups of four: vector loads for x, scalar for y
    for (; j < s.nvec; j += STRIDE) {
      const float4 vx = ld_vec_at(xb, j);
      float4 vy;
      vy.x = Ld<T>::one(yb + 4u * j); vy.y = Ld<T>::one(yb + 4u * j + 1);
      vy.z = Ld<T>::one(yb + 4u * j + 2); vy.w = Ld<T>::one(yb + 4u * j + 3);
      metric_vec<MODE, OFF, CODES>(vx, vy, p, a, CODES ? cb + 4u * j : nullptr);
    }
  }
  if (tid < s.head) {
    metric_elem<MODE, OFF, CODES>(Ld<T>::one(x + tid), PAIR ? Ld<T>::one(y + tid) : 0.0f, p, a[0],
                                  CODES ? codes + tid : nullptr);
  }
  if (tid < s.tail) {
    const uint32_t i = s.head + 4u * s.nvec + tid;
    metric_elem<MODE, OFF, CODES>(Ld<T>::one(x + i), PAIR ? Ld<T>::one(y + i) : 0.0f, p, a[1],
                                  CODES ? codes + i : nullptr);
  }
}

// Parameters of group G as the element arithmetic wants them.  Integer zero point z (scheme 2, the
// offset slot carries z): the arithmetic is the offset-free path on d = q - z -- clamp to
// [-z, top - z], e = x - d*step -- and only the stored code differs (d + z).  Written without
// branches: z is 0 for the other schemes.
__device__ __forceinline__ void load_params(QP& p, const TensorRec* tr, const float* __restrict__ step,
                                            const float* __restrict__ inv, const float* __restrict__ offset,
                                            uint32_t G) {
  const float top = top_code(tr->asym != 0, tr->bits);
  const float qmin0 = tr->asym ? 0.0f : -top;
  const bool zp = tr->asym == 2;
  p.step = __ldg(step + G); p.inv = __ldg(inv + G);
  const float off = __ldg(offset + G);
  const float z = zp ? off : 0.0f;
  p.off = zp ? 0.0f : off;
  p.bias = z; p.qmin = qmin0 - z; p.qmax = top - z;
}

// A tile of whole rows.  Kept out of line: these walkers run for a small share of the bytes (weight
// rows, small feature maps), and inlined into the tile loop they compete with the flat path for
// its registers.  Returns the tile's sums folded into one accumulator.
//
// The metrics are sums over the whole tensor; only the quantization parameters change from row to
// row.  A tile of rows shorter than kPieceRow is therefore streamed like a flat run by the whole CTA
// (16-byte loads, several in flight per thread) and every 16-byte group fetches the parameters of
// the row(s) it lies in; these loads hit L1, since neighbouring groups share a row.  Rows shorter
// than four elements, and pairs whose x and y sit at different offsets inside a 16-byte group,
// are walked one element per thread.
struct RowParams {
  const TensorRec* tr;
  const float* __restrict__ step;
  const float* __restrict__ inv;
  const float* __restrict__ offset;
  uint32_t inner, channels, row0c, gbase;
  float top, qmin0;
  bool zp;
  __device__ __forceinline__ RowParams(const Tile& tl, const TensorRec* t, const float* s, const float* i, const float* o)
      : tr(t), step(s), inv(i), offset(o), inner((uint32_t)t->inner), channels(t->channels),
        row0c((uint32_t)(tl.row0 % t->channels)), gbase(t->group_base), top(top_code(t->asym != 0, t->bits)),
        qmin0(t->asym ? 0.0f : -top_code(false, t->bits)), zp(t->asym == 2) {}
  // parameters of the row that holds element e of the tile (same values as load_params)
  __device__ __forceinline__ QP of_elem(uint32_t e) const { return of_group((row0c + e / inner) % channels); }
  __device__ __forceinline__ QP of_group(uint32_t g) const {
    const uint32_t G = gbase + g;
    QP p;
    p.step = __ldg(step + G); p.inv = __ldg(inv + G);
    const float off = __ldg(offset + G);
    const float z = zp ? off : 0.0f;
    p.off = zp ? 0.0f : off;
    p.bias = z; p.qmin = qmin0 - z; p.qmax = top - z;
    return p;
  }
};

// Rows of 4..kPieceRow-1 elements, x (and y) 16-byte aligned after the same `head` elements: the
// aligned body is walked like a flat run (thread t takes 16-byte groups t, t+256, ...), and every
// thread tracks the row its current group starts in incrementally -- a step of 1024 elements
// advances the row by 1024 / inner and the position in the row by 1024 % inner -- so that no
// division is needed per group.  A group that straddles a row end takes the parameters of both
// rows and picks per element.
template <uint32_t MODE, bool OFF, bool CODES, class T, class ACC>
__device__ __forceinline__ void metric_rows_vec(const T* __restrict__ x, const T* __restrict__ y, uint8_t* codes,
                                                uint32_t count, uint32_t head, const RowParams& rp, ACC* a) {
  constexpr bool PAIR = MODE != kSelf;
  constexpr uint32_t U = PAIR ? 4 : 8;                      // the same bytes in flight as the flat walker
  const uint32_t inner = rp.inner, channels = rp.channels;
  const uint32_t nvec = (count - head) >> 2, tail = (count - head) & 3u;
  const T* xb = x + head;
  const T* yb = PAIR ? y + head : nullptr;
  uint8_t* cb = CODES ? codes + head : nullptr;
  constexpr uint32_t kStep = 4u * kThreads;                    // elements between a thread's consecutive groups
  const uint32_t q = kStep / inner, r = kStep - q * inner;
  uint32_t e = head + 4u * threadIdx.x;                       // index in the tile of the group's first element
  uint32_t rem = e % inner;                                    // its position in its row
  uint32_t g = (rp.row0c + e / inner) % channels;              // the row's group
  for (uint32_t j = threadIdx.x; j < nvec; j += U * kThreads) {          // the last round is clamped: loads in bounds, maybe unused
    float4 vx[U], vy[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      const uint32_t k = min(j + u * kThreads, nvec - 1u);
      vx[u] = ld_vec_at(xb, k);
      if (PAIR) vy[u] = ld_vec_at(yb, k); else vy[u] = vx[u];
    }
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      const uint32_t k = j + u * kThreads;
      if (k < nvec) {
        const QP pa = rp.of_group(g);
        const uint32_t left = inner - rem;                     // elements of this row from the group's first one on
        uint8_t* c = CODES ? cb + 4u * k : nullptr;
        if (left >= 4u) {
          metric_vec<MODE, OFF, CODES>(vx[u], vy[u], pa, a, c);
        } else {                                               // the group ends in the next row (inner >= 4: at most one row end)
          const QP pb = rp.of_group(g + 1u == channels ? 0u : g + 1u);
          metric_elem<MODE, OFF, CODES>(vx[u].x, vy[u].x, pa, a[0], c);
          metric_elem<MODE, OFF, CODES>(vx[u].y, vy[u].y, left > 1u ? pa : pb, a[1], c + 1);
          metric_elem<MODE, OFF, CODES>(vx[u].z, vy[u].z, left > 2u ? pa : pb, a[2], c + 2);
          metric_elem<MODE, OFF, CODES>(vx[u].w, vy[u].w, pb, a[3], c + 3);
        }
        // next group of this thread: kStep elements on
        rem += r; g += q;
        if (rem >= inner) { rem -= inner; ++g; }
        if (g >= channels) g %= channels;
      }
    }
  }
  // the few elements before and after the aligned body, one per thread
  if (threadIdx.x < head + tail) {
    const uint32_t i = threadIdx.x < head ? threadIdx.x : head + 4u * nvec + (threadIdx.x - head);
    const QP p = rp.of_elem(i);
    metric_elem<MODE, OFF, CODES>(Ld<T>::one(x + i), PAIR ? Ld<T>::one(y + i) : 0.0f, p, a[0], CODES ? codes + i : nullptr);
  }
}

template <uint32_t MODE, bool OFF, bool CODES, class T, class ACC>
__device__ __forceinline__ void metric_rows_scalar(const T* __restrict__ x, const T* __restrict__ y, uint8_t* codes,
                                                   uint32_t count, const RowParams& rp, ACC* a) {
  uint32_t e = threadIdx.x;
  for (; e + 3u * kThreads < count; e += 4u * kThreads) {
    float vx[4], vy[4];
#pragma unroll
    for (uint32_t u = 0; u < 4; ++u) {
      vx[u] = Ld<T>::one(x + e + u * kThreads);
      vy[u] = (MODE != kSelf) ? Ld<T>::one(y + e + u * kThreads) : 0.0f;
    }
#pragma unroll
    for (uint32_t u = 0; u < 4; ++u) {
      const uint32_t i = e + u * kThreads;
      const QP p = rp.of_elem(i);
      metric_elem<MODE, OFF, CODES>(vx[u], vy[u], p, a[u], CODES ? codes + i : nullptr);
    }
  }
  for (; e < count; e += kThreads) {
    const QP p = rp.of_elem(e);
    metric_elem<MODE, OFF, CODES>(Ld<T>::one(x + e), (MODE != kSelf) ? Ld<T>::one(y + e) : 0.0f, p, a[0],
                                  CODES ? codes + e : nullptr);
  }
}

// Rows of kPieceRow elements or more: the tile is cut into one contiguous chunk per warp (a multiple
// of four elements); a warp walks its chunk row piece by row piece with the flat walker, fetching
// the row's parameters once per piece.  Eight independent streams whatever the row length.
constexpr uint32_t kPieceRow = 512;

template <uint32_t MODE, bool CODES, class T, class ACC>
__device__ __forceinline__ void metric_rows_pieces(const T* __restrict__ x, const T* __restrict__ y, uint8_t* codes,
                                                   const Tile& tl, const TensorRec* tr,
                                                   const float* __restrict__ step, const float* __restrict__ inv,
                                                   const float* __restrict__ offset, ACC* a) {
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t inner = (uint32_t)tr->inner, channels = tr->channels;
  const uint32_t chunk = (tl.count + 4u * kWarps - 1u) / (4u * kWarps) * 4u;
  uint32_t c0 = min(warp * chunk, tl.count);
  const uint32_t c1 = min(c0 + chunk, tl.count);
  uint32_t row = c0 / inner;
  uint32_t row_end = (row + 1u) * inner;
  uint32_t g = (uint32_t)((tl.row0 + row) % channels);
  QP p;
  while (c0 < c1) {
    const uint32_t p1 = min(c1, row_end);
    load_params(p, tr, step, inv, offset, tr->group_base + g);
    if (MODE == kRaw || p.off == 0.0f)
      metric_flat<MODE, false, CODES, 32>(x + c0, y + c0, codes + c0, p1 - c0, p, a, lane);
    else
      metric_flat<MODE, true, CODES, 32>(x + c0, y + c0, codes + c0, p1 - c0, p, a, lane);
    c0 = p1; row_end += inner;
    if (++g == channels) g = 0;
  }
}

template <uint32_t MODE, bool CODES, class T, class ACC>
__device__ __noinline__ ACC metric_rows(Tile tl, const TensorRec* tr, const float* __restrict__ step,
                                        const float* __restrict__ inv, const float* __restrict__ offset,
                                        uint8_t* codes_base, ACC seed) {
  const T* x = reinterpret_cast<const T*>(tr->x) + tl.begin;
  const T* y = (MODE != kSelf) ? reinterpret_cast<const T*>(tr->y) + tl.begin : nullptr;
  uint8_t* codes = CODES ? codes_base + tl.begin : nullptr;
  ACC a[4] = {seed, seed, seed, seed};
  if (tr->inner >= kPieceRow) {
    metric_rows_pieces<MODE, CODES>(x, y, codes, tl, tr, step, inv, offset, a);
    return ACC::fold(a);
  }
  const RowParams rp(tl, tr, step, inv, offset);
  // elements up to the first 16-byte boundary of x; the vector walker needs y at the same phase
  const uint32_t head = min((4u - (uint32_t)(((uintptr_t)x / sizeof(T)) & 3u)) & 3u, tl.count);
  constexpr uintptr_t kVecMask = 4u * sizeof(T) - 1u;
  const bool vec = rp.inner >= 4u && tl.count - head >= 4u &&
                   (MODE == kSelf || (((uintptr_t)(y + head)) & kVecMask) == 0);
  // a real-valued offset needs the form of the arithmetic that splits x - offset exactly; with a
  // zero offset both forms give the same value
  const bool off = MODE != kRaw && tr->asym == 1;
  if (vec) {
    if (off) metric_rows_vec<MODE, MODE != kRaw, CODES>(x, y, codes, tl.count, head, rp, a);
    else metric_rows_vec<MODE, false, CODES>(x, y, codes, tl.count, head, rp, a);
  } else {
    if (off) metric_rows_scalar<MODE, MODE != kRaw, CODES>(x, y, codes, tl.count, rp, a);
    else metric_rows_scalar<MODE, false, CODES>(x, y, codes, tl.count, rp, a);
  }
  return ACC::fold(a);
}

template <uint32_t MODE, bool CODES, class T, class ACC>
__device__ __forceinline__ void metric_tile_typed(const Tile& tl, const TensorRec* tr,
                                                  const float* __restrict__ step, const float* __restrict__ inv,
                                                  const float* __restrict__ offset, uint8_t* codes_base, ACC* a) {
  if (tl.rows == 0) {
    const T* x = reinterpret_cast<const T*>(tr->x) + tl.begin;
    const T* y = (MODE != kSelf) ? reinterpret_cast<const T*>(tr->y) + tl.begin : nullptr;
    uint8_t* codes = CODES ? codes_base + tl.begin : nullptr;
    QP p;
    load_params(p, tr, step, inv, offset, tr->group_base + (uint32_t)tl.row0);
    if (MODE == kRaw || p.off == 0.0f) metric_flat<MODE, false, CODES>(x, y, codes, tl.count, p, a);
    else metric_flat<MODE, true, CODES>(x, y, codes, tl.count, p, a);
  } else {
    a[0].merge(metric_rows<MODE, CODES, T>(tl, tr, step, inv, offset, codes_base, a[0].fresh()));
  }
}

// Dispatch on the element type of the tensor (compiled out when ANY16 is false: all binary32).
template <uint32_t MODE, bool CODES, bool ANY16 = true, class ACC>
__device__ __forceinline__ void metric_tile(const Tile& tl, const TensorRec* tr,
                                            const float* __restrict__ step, const float* __restrict__ inv,
                                            const float* __restrict__ offset, uint8_t* codes_base, ACC* a) {
  if (!ANY16 || tr->dtype == kF32) metric_tile_typed<MODE, CODES, float>(tl, tr, step, inv, offset, codes_base, a);
  else if (tr->dtype == kF16) metric_tile_typed<MODE, CODES, __half>(tl, tr, step, inv, offset, codes_base, a);
  else metric_tile_typed<MODE, CODES, __nv_bfloat16>(tl, tr, step, inv, offset, codes_base, a);
}

// Slot of (tensor, CTA): the CTAs that own tiles of a tensor are numbered in the order of the
// tensor's first tiles, rank = (b - tile_first) mod grid < min(grid, tiles of the tensor).
__device__ __forceinline__ uint32_t slot_of(const TensorRec* tr) {
  const uint32_t g = gridDim.x;
  const uint32_t rank = (blockIdx.x + g - tr->tile_first % g) % g;
  return tr->slot_first + rank;
}

// Folds one tensor once every CTA that owns a tile of it has written its slot: fixed-order
// binary64 sum of the tensor's slots, then MSE (Eq. 7), SQNR (Eq. 6) and, when asked for, the
// cosine similarity (Eq. 8) between the reference tensor A = x and the compared tensor B = x - e:
// A.B = sig - xe, |B|^2 = sig - 2 xe + sse.  Runs in the CTA that drew the tensor's last ticket
// (CTA 0 for a tensor without elements); the slots, written by other CTAs, are read through L2.
template <bool COS>
__device__ __noinline__ void metrics_fold_tensor(const MetricsArgs& a, uint32_t t) {
  __shared__ double sh_e[kThreads], sh_s[kThreads], sh_x[COS ? kThreads : 1];
  const TensorRec tr = a.tensors[t];
  const uint32_t tid = threadIdx.x;
  double e = 0.0, s = 0.0, xe = 0.0;
  for (uint32_t k = tid; k < tr.metrics_ctas; k += kThreads) {
    const double2 p = __ldcg(a.partials + tr.slot_first + k);
    e = __dadd_rn(e, p.x);
    s = __dadd_rn(s, p.y);
    if (COS) xe = __dadd_rn(xe, __ldcg(a.partials_xe + tr.slot_first + k));
  }
  sh_e[tid] = e; sh_s[tid] = s;
  if (COS) sh_x[tid] = xe;
  __syncthreads();
  for (uint32_t o = kThreads / 2; o > 0; o >>= 1) {
    if (tid < o) {
      sh_e[tid] = __dadd_rn(sh_e[tid], sh_e[tid + o]);
      sh_s[tid] = __dadd_rn(sh_s[tid], sh_s[tid + o]);
      if (COS) sh_x[tid] = __dadd_rn(sh_x[tid], sh_x[tid + o]);
    }
    __syncthreads();
  }
  if (tid == 0) {
    const double sse = sh_e[0], sig = sh_s[0];
    const double inf = __longlong_as_double(0x7ff0000000000000ll);
    a.sse[t] = sse;
    a.sig[t] = sig;
    a.mse[t] = tr.n_elems ? __ddiv_rn(sse, (double)tr.n_elems) : 0.0;
    double q;
    if (sse == 0.0) q = inf;
    else if (sig == 0.0) q = -inf;
    else q = __dmul_rn(10.0, log10(__ddiv_rn(sig, sse)));
    a.sqnr_db[t] = q;
    if (COS) {
      const double ab = sig - sh_x[0];
      const double bb = sig - 2.0 * sh_x[0] + sse;
      const double den = sqrt(sig) * sqrt(bb > 0.0 ? bb : 0.0);
      a.cosine[t] = den > 0.0 ? ab / den : 0.0;       // a zero vector has no direction
    }
    a.tickets[t] = 0u;                                // ready for the next pass
  }
  __syncthreads();                                    // the shared arrays may be reused by the next fold
}

// COS adds the sum x*e (third slot array) needed for the cosine similarity.  FOLD = true: the CTA
// that finishes a tensor last folds its slots; FOLD = false: metrics_fold_kernel follows, and the
// main loop carries neither the fold code nor a fence.
template <bool COS, bool ANY16, bool FOLD>
__global__ void __launch_bounds__(kThreads, 3)       // 4 CTAs per SM did not run faster
metrics_kernel(const __grid_constant__ MetricsArgs a, const TensorRec* __restrict__ tensors,
               const Tile* __restrict__ tiles, uint32_t n_tiles, uint32_t scan_begin, uint32_t scan_end) {
  using ACC = typename std::conditional<COS, AccCos, Acc>::type;
  constexpr uint32_t kNone = 0xffffffffu;
  __shared__ double sh_w[3][kWarps];
  __shared__ uint32_t s_last;
  const float* __restrict__ step = a.step;
  const float* __restrict__ inv = a.inv;
  const float* __restrict__ offset = a.offset;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  dependency_wait();
  // tensors without elements are owned by no CTA: CTA 0 folds them
  if (FOLD && blockIdx.x == 0)
    for (uint32_t t = scan_begin; t < scan_end; ++t)
      if (tensors[t].metrics_ctas == 0) metrics_fold_tensor<COS>(a, t);
  uint32_t cur = kNone;
  uint32_t owed = kNone, drawn = 0; // FOLD: the tensor before cur and the ticket thread 0 drew for it
  double run_sse = 0.0, run_sig = 0.0, run_xe = 0.0;
  // Ticket protocol of the fused fold: right after its slot store thread 0 fences and draws the
  // tensor's ticket without looking at the result; the CTA looks at it at its next tensor
  // boundary and folds the tensor if the ticket was the last one.  The atomic's round trip hides
  // behind the next tensor's stream; nobody waits for another CTA.
  auto settle = [&](uint32_t t) {
    if (threadIdx.x == 0) {
      const bool last = drawn == tensors[t].metrics_ctas - 1u;
      if (last) __threadfence();
      s_last = last;
    }
    __syncthreads();
    if (s_last) metrics_fold_tensor<COS>(a, t);
  };
  // The CTA is done with tensor t: lanes fold by a fixed butterfly, warps in warp order, one
  // {sum e^2, sum x^2} pair goes to the CTA's own slot.
  auto flush = [&](uint32_t t) {
    if (FOLD && owed != kNone) settle(owed);
    const TensorRec* tr = tensors + t;
    const double sse = warp_sum_f64(run_sse), sig = warp_sum_f64(run_sig);
    double xe = 0.0;
    if (COS) xe = warp_sum_f64(run_xe);
    if (lane == 0) { sh_w[0][warp] = sse; sh_w[1][warp] = sig; if (COS) sh_w[2][warp] = xe; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double e = sh_w[0][0], s = sh_w[1][0], x = COS ? sh_w[2][0] : 0.0;
#pragma unroll
      for (int w = 1; w < kWarps; ++w) {
        e = __dadd_rn(e, sh_w[0][w]); s = __dadd_rn(s, sh_w[1][w]);
        if (COS) x = __dadd_rn(x, sh_w[2][w]);
      }
      const uint32_t slot = slot_of(tr);
      a.partials[slot] = make_double2(e, s);
      if (COS) a.partials_xe[slot] = x;
      if (FOLD) {
        __threadfence();                               // the slot is visible before the ticket is
        drawn = atomicAdd(a.tickets + t, 1u);
      }
    }
    __syncthreads();                                   // sh_w may be rewritten by the next flush
    owed = t;
  };
  for (uint32_t ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
    const Tile tl = load_tile(tiles, ti);
    const TensorRec* tr = tensors + tl.tensor;
    if (tl.tensor != cur) {
      if (cur != kNone) flush(cur);
      cur = tl.tensor; run_sse = 0.0; run_sig = 0.0; run_xe = 0.0;
    }
    ACC acc[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[k].clear();
    const uint32_t mode = tr->pair_mode;
    uint8_t* cbase = a.codes ? a.codes[tl.tensor] : nullptr;
    const bool codes = cbase != nullptr && mode != kRaw;
    if (mode == kSelf) {
      if (codes) metric_tile<kSelf, true, ANY16>(tl, tr, step, inv, offset, cbase, acc);
      else metric_tile<kSelf, false, ANY16>(tl, tr, step, inv, offset, nullptr, acc);
    } else if (mode == kRequant) {
      if (codes) metric_tile<kRequant, true, ANY16>(tl, tr, step, inv, offset, cbase, acc);
      else metric_tile<kRequant, false, ANY16>(tl, tr, step, inv, offset, nullptr, acc);
    } else {
      metric_tile<kRaw, false, ANY16>(tl, tr, step, inv, offset, nullptr, acc);
    }
    // this lane's tile sums in binary32 with a fixed association, then into the binary64 totals
    const float sse = __fadd_rn(__fadd_rn(acc[0].sse, acc[1].sse), __fadd_rn(acc[2].sse, acc[3].sse));
    const float sig = __fadd_rn(__fadd_rn(acc[0].sig, acc[1].sig), __fadd_rn(acc[2].sig, acc[3].sig));
    run_sse = __dadd_rn(run_sse, (double)sse);
    run_sig = __dadd_rn(run_sig, (double)sig);
    if constexpr (COS) {
      const float xe = __fadd_rn(__fadd_rn(acc[0].xe, acc[1].xe), __fadd_rn(acc[2].xe, acc[3].xe));
      run_xe = __dadd_rn(run_xe, (double)xe);
    }
  }
  allow_dependents();            // this CTA has issued all its loads: the next kernel may start to launch
  if (cur != kNone) {
    flush(cur);
    if (FOLD) settle(cur);
  }
}

// One CTA per tensor of the stage: the fold, for stages whose streaming kernel does not fold.
template <bool COS>
__global__ void __launch_bounds__(kThreads)
metrics_fold_kernel(const __grid_constant__ MetricsArgs a, uint32_t tensor_begin) {
  allow_dependents();
  dependency_wait();
  metrics_fold_tensor<COS>(a, tensor_begin + blockIdx.x);
}

// ------------------------------------------------------------------------------------------------
// KL divergence (Eq. 9) between the distribution of x and that of the tensor it is compared with,
// both binned on kKlBins linear bins of |value| over [0, absmax of x].  Same tile walk and
// quantizer as the metrics kernel; the accumulator bins instead of summing.  Each warp owns a
// private pair of histograms in shared memory; they are merged into the 64-bit global ones when
// the CTA moves to another tensor.  Counts are integers: the result does not depend on order.
constexpr uint32_t kKlBins = QV2_KL_BINS;

struct AccKL {
  static constexpr bool kWantsB = true;
  uint32_t* hp;      // this warp's histogram of |x|
  uint32_t* hq;      // ... and of |b|
  float w;           // fl(kKlBins / absmax)
  __device__ __forceinline__ static uint32_t bin(float v, float w) {
    const float f = __fmul_rn(fabsf(v), w);
    const uint32_t b = __float_as_uint(__fadd_rz(f, 8388608.0f)) - 0x4B000000u;   // trunc for 0 <= f < 2^23
    return min(b, kKlBins - 1u);
  }
  __device__ __forceinline__ void add_b(float x, float b) {
    if (!isfinite(x) || !isfinite(b)) return;
    atomicAdd(hp + bin(x, w), 1u);
    atomicAdd(hq + bin(b, w), 1u);
  }
  // the counts live in shared memory: a copy counts into the same histograms
  __device__ __forceinline__ AccKL fresh() const { return *this; }
  __device__ __forceinline__ static AccKL fold(const AccKL* a) { return a[0]; }
  __device__ __forceinline__ void merge(const AccKL&) {}
};

__global__ void __launch_bounds__(kThreads, 2)
kl_kernel(const TensorRec* __restrict__ tensors, const Tile* __restrict__ tiles, uint32_t n_tiles,
          const float* __restrict__ step, const float* __restrict__ inv, const float* __restrict__ offset,
          const float* __restrict__ tensor_absmax, unsigned long long* hists) {
  __shared__ uint32_t sh[kWarps * 2 * kKlBins];
  constexpr uint32_t kNone = 0xffffffffu;
  const uint32_t warp = threadIdx.x >> 5;
  for (uint32_t b = threadIdx.x; b < kWarps * 2 * kKlBins; b += kThreads) sh[b] = 0;
  __syncthreads();
  uint32_t cur = kNone, since_flush = 0;
  float w = 0.0f;
  for (uint32_t ti = blockIdx.x;; ti += gridDim.x) {
    const bool more = ti < n_tiles;
    Tile tl;
    if (more) tl = load_tile(tiles, ti);
    if (cur != kNone && (!more || tl.tensor != cur || since_flush >= 16384u)) {
      __syncthreads();                               // every warp is done with its last tile
      unsigned long long* h = hists + (size_t)cur * 2 * kKlBins;
      for (uint32_t b = threadIdx.x; b < kWarps * 2 * kKlBins; b += kThreads) {
        const uint32_t c = sh[b];
        if (c) { atomicAdd(h + (b % (2 * kKlBins)), (unsigned long long)c); sh[b] = 0; }
      }
      __syncthreads();
      since_flush = 0;
    }
    if (!more) break;
    const TensorRec* tr = tensors + tl.tensor;
    if (tl.tensor != cur) {
      cur = tl.tensor;
      const float A = tensor_absmax[cur];
      w = (A > 0.0f) ? __fdiv_rn((float)kKlBins, A) : 0.0f;
      if (!isfinite(w)) w = 0.0f;
    }
    AccKL a[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) { a[k].hp = sh + warp * 2 * kKlBins; a[k].hq = a[k].hp + kKlBins; a[k].w = w; }
    const uint32_t mode = tr->pair_mode;
    if (mode == kSelf) metric_tile<kSelf, false>(tl, tr, step, inv, offset, nullptr, a);
    else if (mode == kRequant) metric_tile<kRequant, false>(tl, tr, step, inv, offset, nullptr, a);
    else metric_tile<kRaw, false>(tl, tr, step, inv, offset, nullptr, a);
    ++since_flush;
  }
}

// One CTA per tensor: the tensor-wide absmax from the per-group values.
__global__ void __launch_bounds__(256)
tensor_absmax_kernel(const TensorRec* __restrict__ tensors, const float* __restrict__ gabsmax, float* out) {
  __shared__ float red[256];
  const TensorRec tr = tensors[blockIdx.x];
  float m = 0.0f;
  for (uint32_t g = threadIdx.x; g < tr.n_groups; g += 256) m = fmaxf(m, gabsmax[tr.group_base + g]);
  red[threadIdx.x] = m;
  __syncthreads();
  for (uint32_t o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + o]);
    __syncthreads();
  }
  if (threadIdx.x == 0) out[blockIdx.x] = red[0];
}

// One thread per tensor: add-one smoothing, then the sum in bin order.
__global__ void kl_finalize_kernel(uint32_t n, const unsigned long long* __restrict__ hists, double* kl_out) {
  const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const unsigned long long* hp = hists + (size_t)t * 2 * kKlBins;
  const unsigned long long* hq = hp + kKlBins;
  unsigned long long cnt = 0;
  for (uint32_t j = 0; j < kKlBins; ++j) cnt += hp[j];
  const double den = __dadd_rn((double)cnt, (double)kKlBins);
  double kl = 0.0;
  for (uint32_t j = 0; j < kKlBins; ++j) {
    const double p = __ddiv_rn(__dadd_rn((double)hp[j], 1.0), den);
    const double q = __ddiv_rn(__dadd_rn((double)hq[j], 1.0), den);
    kl = __dadd_rn(kl, __dmul_rn(p, log(__ddiv_rn(p, q))));
  }
  kl_out[t] = kl;
}

}  // namespace

uint32_t metrics_grid_cap(int sm_count, bool fused) {
  int cache = 0;
  const void* k = fused ? (const void*)metrics_kernel<false, false, true> : (const void*)metrics_kernel<false, false, false>;
  return (uint32_t)persistent_grid(k, &cache, sm_count, 0x7fffffffu);
}
uint32_t kl_grid_cap(int sm_count) {
  int cache = 0;
  return (uint32_t)persistent_grid((const void*)kl_kernel, &cache, sm_count, 0x7fffffffu);
}

cudaError_t launch_metrics(const Launch& l, const Stage& st, bool any16, const Tile* tiles, const MetricsArgs& a) {
  const uint32_t n_tiles = st.tile_end - st.tile_begin;
  const Tile* tp = tiles + st.tile_begin;
  const bool fold = st.fused_fold;
  const uint32_t s0 = fold && st.any_empty ? st.tensor_begin : 0u, s1 = fold && st.any_empty ? st.tensor_end : 0u;
#define QV2_LAUNCH_METRICS(COS, A16, FOLD) \
  e = launch_kernel(l, metrics_kernel<COS, A16, FOLD>, st.metrics_grid, kThreads, a, a.tensors, tp, n_tiles, s0, s1)
#define QV2_LAUNCH_METRICS_F(COS, A16) do { if (fold) QV2_LAUNCH_METRICS(COS, A16, true); else if (n_tiles) QV2_LAUNCH_METRICS(COS, A16, false); } while (0)
  cudaError_t e = cudaSuccess;
  if (a.cosine) { if (any16) QV2_LAUNCH_METRICS_F(true, true); else QV2_LAUNCH_METRICS_F(true, false); }
  else { if (any16) QV2_LAUNCH_METRICS_F(false, true); else QV2_LAUNCH_METRICS_F(false, false); }
#undef QV2_LAUNCH_METRICS_F
#undef QV2_LAUNCH_METRICS
  if (e != cudaSuccess || fold) return e;
  const uint32_t nt = st.tensor_end - st.tensor_begin;
  return a.cosine ? launch_kernel(l, metrics_fold_kernel<true>, nt, kThreads, a, st.tensor_begin)
                  : launch_kernel(l, metrics_fold_kernel<false>, nt, kThreads, a, st.tensor_begin);
}

cudaError_t launch_kl(const Launch& l, uint32_t grid_cap, const TensorRec* tensors, uint32_t n_tensors,
                      const Tile* tiles, uint32_t n_tiles, const float* step, const float* inv,
                      const float* offset, const float* gabsmax, float* tensor_absmax,
                      unsigned long long* hists, double* kl) {
  tensor_absmax_kernel<<<n_tensors, 256, 0, l.stream>>>(tensors, gabsmax, tensor_absmax);
  if (n_tiles) {
    const uint32_t grid = grid_cap < n_tiles ? (grid_cap ? grid_cap : 1u) : n_tiles;
    kl_kernel<<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, step, inv, offset, tensor_absmax, hists);
  }
  kl_finalize_kernel<<<(n_tensors + 63) / 64, 64, 0, l.stream>>>(n_tensors, hists, kl);
  return cudaGetLastError();
}

}  // namespace qv2

// ================================================================================================
// qv2_quant_metrics_noalloc: the fused fake-quantize + error reduction for ONE tensor with no
// allocation of any kind.  Its partial sums live in a fixed array inside the loaded library image
// instead of context scratch, and the tensor is described to the kernel by value instead of
// through uploaded tables.  The per-element arithmetic is the code above, unchanged.
// ================================================================================================
namespace qv2 {
namespace {

// One {sum e^2, sum x^2} pair per warp and tile.  1 MiB per GPU that loads the library, held
// until the process exits.  Every slot a call reads is written by that same call first, so the
// array needs no clearing between calls; it does keep the previous call's contents.
constexpr uint32_t kNoAllocMaxTiles = QV2_NOALLOC_MAX_ELEMS / kTileElems;
static __device__ __align__(256) double2 g_noalloc_slots[kNoAllocMaxTiles * kWarps];

struct NoAllocJob {
  TensorRec tr;
  uint64_t rows;            // outer * channels
  uint32_t n_tiles;
  uint32_t cut;             // 0: flat run, 1: long rows cut at row boundaries, 2: whole short rows
  uint32_t tiles_per_row;   // cut 1
  uint32_t rows_per_tile;   // cut 2
};

// The same decomposition as the host planner, evaluated on the fly for one tensor.
__device__ __forceinline__ Tile noalloc_tile(const NoAllocJob& j, uint32_t ti) {
  Tile t;
  t.tensor = 0; t.pack = 0;
  if (j.cut == 0) {
    t.begin = (uint64_t)ti * kTileElems;
    const uint64_t left = j.tr.n_elems - t.begin;
    t.count = left > kTileElems ? kTileElems : (uint32_t)left;
    t.row0 = 0; t.rows = 0;
  } else if (j.cut == 1) {
    const uint64_t row = ti / j.tiles_per_row;
    const uint64_t piece = ti % j.tiles_per_row;
    t.begin = row * j.tr.inner + piece * kTileElems;
    const uint64_t left = j.tr.inner - piece * kTileElems;
    t.count = left > kTileElems ? kTileElems : (uint32_t)left;
    t.row0 = row % j.tr.channels; t.rows = 0;
  } else {
    const uint64_t row = (uint64_t)ti * j.rows_per_tile;
    const uint64_t left = j.rows - row;
    t.rows = left > j.rows_per_tile ? j.rows_per_tile : (uint32_t)left;
    t.begin = row * j.tr.inner; t.row0 = row;
    t.count = (uint32_t)(t.rows * j.tr.inner);
  }
  return t;
}

__global__ void __launch_bounds__(kThreads, 4)
metrics_noalloc_kernel(const __grid_constant__ NoAllocJob job, const float* __restrict__ step,
                       const float* __restrict__ inv, const float* __restrict__ offset,
                       double2* __restrict__ slots) {
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const TensorRec* tr = &job.tr;
  for (uint32_t ti = blockIdx.x; ti < job.n_tiles; ti += gridDim.x) {
    const Tile tl = noalloc_tile(job, ti);
    Acc a[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) a[k].clear();
    if (tr->pair_mode == kSelf) metric_tile<kSelf, false>(tl, tr, step, inv, offset, nullptr, a);
    else if (tr->pair_mode == kRequant) metric_tile<kRequant, false>(tl, tr, step, inv, offset, nullptr, a);
    else metric_tile<kRaw, false>(tl, tr, step, inv, offset, nullptr, a);
    float sse = __fadd_rn(__fadd_rn(a[0].sse, a[1].sse), __fadd_rn(a[2].sse, a[3].sse));
    float sig = __fadd_rn(__fadd_rn(a[0].sig, a[1].sig), __fadd_rn(a[2].sig, a[3].sig));
    sse = warp_sum(sse);
    sig = warp_sum(sig);
    if (lane == 0) slots[(size_t)ti * kWarps + warp] = make_double2((double)sse, (double)sig);
  }
}

// One CTA: fixed-order binary64 sum of the n_tiles * kWarps slots, then MSE and SQNR.
__global__ void __launch_bounds__(1024)
metrics_noalloc_finalize_kernel(uint32_t n_slots, uint64_t n_elems, const double2* __restrict__ slots,
                                double* out4) {
  __shared__ double sh_e[1024], sh_s[1024];
  double e = 0.0, s = 0.0;
  for (uint32_t k = threadIdx.x; k < n_slots; k += 1024) {
    const double2 p = slots[k];
    e = __dadd_rn(e, p.x);
    s = __dadd_rn(s, p.y);
  }
  sh_e[threadIdx.x] = e; sh_s[threadIdx.x] = s;
  __syncthreads();
  for (uint32_t o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      sh_e[threadIdx.x] = __dadd_rn(sh_e[threadIdx.x], sh_e[threadIdx.x + o]);
      sh_s[threadIdx.x] = __dadd_rn(sh_s[threadIdx.x], sh_s[threadIdx.x + o]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double sse = sh_e[0], sig = sh_s[0];
    const double inf = __longlong_as_double(0x7ff0000000000000ll);
    out4[0] = sse;
    out4[1] = sig;
    out4[2] = n_elems ? __ddiv_rn(sse, (double)n_elems) : 0.0;
    out4[3] = sse == 0.0 ? inf : (sig == 0.0 ? -inf : __dmul_rn(10.0, log10(__ddiv_rn(sig, sse))));
  }
}

// Per-device set-up state.  The array's name is only a handle on the host; its device address
// has to be asked for, once per device, with that device current.
constexpr int kMaxDevices = 64;
struct NoAllocDevice {
  std::once_flag once;
  double2* slots = nullptr;     // null until the set-up has succeeded
  int grid_cap = 1;
};
NoAllocDevice g_noalloc_dev[kMaxDevices];

}  // namespace
}  // namespace qv2

extern "C" int qv2_quant_metrics_noalloc(int device, void* stream, const qv2_tensor_desc* desc,
                                         const float* step, const float* inv, const float* offset,
                                         double* result4) {
  using namespace qv2;
  if (!desc || !step || !inv || !offset || !result4) return QV2_ERR_NULL;
  if (device < 0 || device >= kMaxDevices) return QV2_ERR_ARG;
  const qv2_tensor_desc& d = *desc;
  if (d.granularity > QV2_PER_CHANNEL || d.scheme > QV2_ASYM_U8_ZP || d.range > QV2_PERCENTILE_GROUP)
    return QV2_ERR_ARG;
  if (d.flags & ~(uint32_t)(QV2_PAIR_RAW | QV2_BITS_MASK)) return QV2_ERR_ARG;   // no code output here
  if (QV2_DESC_BITS(d.flags) < 2 || QV2_DESC_BITS(d.flags) > 16) return QV2_ERR_ARG;
  if ((d.flags & QV2_PAIR_RAW) && !d.y) return QV2_ERR_ARG;
  if (d.channels >= (1ull << 32)) return QV2_ERR_SIZE;
  // sizes: reject anything whose partial sums would not fit the fixed array
  if (d.outer && d.channels > QV2_NOALLOC_MAX_ELEMS / d.outer) return QV2_ERR_SIZE;
  const uint64_t rows = d.outer * d.channels;
  if (rows && d.inner > QV2_NOALLOC_MAX_ELEMS / rows) return QV2_ERR_SIZE;
  const uint64_t ne = rows * d.inner;
  if (ne > 0 && !d.x) return QV2_ERR_NULL;
  if (((uintptr_t)d.x & 3u) || ((uintptr_t)d.y & 3u)) return QV2_ERR_ALIGN;

  NoAllocJob job{};                      // every field the kernel does not use reads zero
  job.tr.x = d.x; job.tr.y = d.y;
  job.tr.n_elems = ne; job.tr.inner = d.inner; job.tr.channels = (uint32_t)d.channels;
  job.tr.per_channel = d.granularity == QV2_PER_CHANNEL;
  job.tr.n_groups = job.tr.per_channel ? (uint32_t)d.channels : 1u;
  job.tr.asym = d.scheme;
  job.tr.range_mode = d.range;
  job.tr.pair_mode = !d.y ? kSelf : ((d.flags & QV2_PAIR_RAW) ? kRaw : kRequant);
  job.tr.percentile = d.percentile;
  job.tr.bits = QV2_DESC_BITS(d.flags);
  job.tr.dtype = kF32;                  // this entry point takes binary32 tensors only
  job.rows = rows; job.tiles_per_row = 1; job.rows_per_tile = 1;
  uint64_t n_tiles;
  if (!job.tr.per_channel || ne == 0) {
    job.cut = 0;
    n_tiles = (ne + kTileElems - 1) / kTileElems;
  } else if (d.inner >= 4096) {          // this entry point keeps its own cut: long rows at row boundaries
    job.cut = 1;
    job.tiles_per_row = (uint32_t)((d.inner + kTileElems - 1) / kTileElems);
    n_tiles = rows * job.tiles_per_row;
  } else {
    job.cut = 2;
    job.rows_per_tile = (uint32_t)(kTileElems / d.inner);
    n_tiles = (rows + job.rows_per_tile - 1) / job.rows_per_tile;
  }
  if (n_tiles > kNoAllocMaxTiles) return QV2_ERR_SIZE;     // ragged rows can need more tiles than N/16384
  job.n_tiles = (uint32_t)n_tiles;

  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return QV2_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return QV2_ERR_CUDA;
  int status = QV2_OK;
  NoAllocDevice& nd = g_noalloc_dev[device];
  // first call on this device: resolve the array's address; host threads racing here run it once
  std::call_once(nd.once, [&]() {
    double2* p = nullptr;
    int sms = 0, per_sm = 0;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_slots) != cudaSuccess || !p ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
      return;                                   // nd.slots stays null: every call reports QV2_ERR_CUDA
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void*)metrics_noalloc_kernel,
                                                      kThreads, 0) != cudaSuccess || per_sm < 1)
      per_sm = 1;
    nd.grid_cap = per_sm * (sms > 0 ? sms : 1);
    nd.slots = p;
  });
  if (!nd.slots) {
    (void)cudaGetLastError();                   // the failed set-up call must not poison later launches
    status = QV2_ERR_CUDA;
  }
  if (status == QV2_OK) {
    cudaStream_t s = (cudaStream_t)stream;
    if (job.n_tiles) {
      const uint32_t grid = job.n_tiles < (uint32_t)nd.grid_cap ? job.n_tiles : (uint32_t)nd.grid_cap;
      metrics_noalloc_kernel<<<grid, kThreads, 0, s>>>(job, step, inv, offset, nd.slots);
      if (cudaPeekAtLastError() != cudaSuccess) { (void)cudaGetLastError(); status = QV2_ERR_CUDA; }
    }
    if (status == QV2_OK) {
      metrics_noalloc_finalize_kernel<<<1, 1024, 0, s>>>(job.n_tiles * kWarps, ne, nd.slots, result4);
      if (cudaPeekAtLastError() != cudaSuccess) { (void)cudaGetLastError(); status = QV2_ERR_CUDA; }
    }
  }
  if (prev != device) cudaSetDevice(prev);
  return status;
}

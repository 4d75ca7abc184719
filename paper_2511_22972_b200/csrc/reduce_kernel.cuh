// Row reduction of the FLy verification step: one streaming pass over a piece
// of a logits row yields the running maximum, the softmax normaliser, the
// weighted sum that gives the entropy (Eq. 5) and the greedy token (Eq. 1).
//
// Work decomposition: unit = (row, split).  One thread block reduces one unit
// and writes one 16-byte Partial.  Inside the block every warp streams its own
// interleaved slices with 128-bit loads, UNROLL loads in flight per lane; the
// warp keeps ONE reference exponent (its running maximum), so a slice costs one
// warp-wide max (redux.sync) and the rescale / index search only runs when the
// maximum actually moves (a handful of times per row).  Per element the steady
// state is: widen, one FMA into the base-2 exponent, one MUFU ex2, two
// accumulations.
#pragma once
#include "fly_common.cuh"
#include "scan_kernel.cuh"

namespace fly {

constexpr int kReduceThreads = 256;
constexpr int kReduceWarps = kReduceThreads / 32;

// Per-warp streaming state.  S/u are per-lane (two accumulator pairs for ILP),
// everything else is warp-uniform.
struct WarpAcc {
  float cur_max;  // raw running maximum (warp-uniform)
  float r;        // cur_max * log2(e): reference exponent of S and u
  int best_idx;   // lowest index holding cur_max (warp-uniform)
  float S0, u0, S1, u1;
};

__device__ __forceinline__ void acc_init(WarpAcc& a) {
  a.cur_max = kMaskFloor;
  a.r = kMaskFloor * kLog2e;
  a.best_idx = kIdxNone;
  a.S0 = a.u0 = a.S1 = a.u1 = 0.f;
}

// Moves the reference exponent to a larger maximum (warp-uniform call).
__device__ __forceinline__ void acc_rebase(WarpAcc& a, float new_max) {
  const float nr = new_max * kLog2e;
  const float d = a.r - nr;  // < 0, finite
  const float sc = ex2_approx(d);
  a.u0 = sc * fmaf(d, a.S0, a.u0);
  a.u1 = sc * fmaf(d, a.S1, a.u1);
  a.S0 *= sc;
  a.S1 *= sc;
  a.r = nr;
  a.cur_max = new_max;
}

__device__ __forceinline__ void acc_add(float x, float nr, float& S, float& u) {
  const float t = fmaf(x, kLog2e, nr);  // nr = -r
  const float e = ex2_approx(t);
  S += e;
  u = fmaf(e, t, u);
}

// ---------------------------------------------------------------------------
// Vector path: rows whose base, stride and length are multiples of 16 bytes.
// A "segment" is one 16-byte load: 8 bf16 or 4 fp32 logits.
// ---------------------------------------------------------------------------

template <typename T> struct Seg;
template <> struct Seg<__nv_bfloat16> { static constexpr int kElems = 8; };
template <> struct Seg<float> { static constexpr int kElems = 4; };

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint32_t bf2_max(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf2_max_nan(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

constexpr uint32_t kNegInf2 = 0xff80ff80u;  // bf16 (-inf, -inf)

// Folds one warp slice of UNROLL*32 segments of bf16 logits, already in registers, into the
// warp's running state.  w[j] is segment seg0 + j*32 + lane of the row (8 logits).
template <int UNROLL>
__device__ __forceinline__ void fold_slice_bf16(WarpAcc& a, uint32_t (&w)[UNROLL][4], int seg0, int lane) {
  constexpr uint32_t kFloor2 = 0xc974c974u;   // bf16(kMaskFloor) twice
  // clamp masked entries to the floor (NaN survives the clamp and ends in S)
  uint32_t lm2 = kFloor2;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      w[j][c] = bf2_max_nan(w[j][c], kFloor2);
      lm2 = bf2_max(lm2, w[j][c]);
    }
  const float lm = fmaxf(bf16lo(lm2), bf16hi(lm2));
  const float wm = warp_max_f32(lm);
  if (wm > a.cur_max) {  // warp-uniform, rare after the first slices
    acc_rebase(a, wm);
    uint32_t first = 0xffffffffu;
    if (lm == wm) {
#pragma unroll
      for (int j = UNROLL - 1; j >= 0; --j)
#pragma unroll
        for (int c = 3; c >= 0; --c) {
          const uint32_t base = (uint32_t)(seg0 + j * 32 + lane) * 8u + (uint32_t)c * 2u;
          if (bf16hi(w[j][c]) == wm) first = base + 1u;
          if (bf16lo(w[j][c]) == wm) first = base;
        }
    }
    a.best_idx = (int)warp_min_u32(first);
  }
  const float nr = -a.r;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      acc_add(bf16lo(w[j][c]), nr, a.S0, a.u0);
      acc_add(bf16hi(w[j][c]), nr, a.S1, a.u1);
    }
}


// The same for fp32 logits: x[j] is segment seg0 + j*32 + lane of the row (4 logits).
template <int UNROLL>
__device__ __forceinline__ void fold_slice_f32(WarpAcc& a, float (&x)[UNROLL][4], int seg0, int lane) {
  float lm = kMaskFloor;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      x[j][c] = max_nan_f32(x[j][c], kMaskFloor);
      lm = fmaxf(lm, x[j][c]);
    }
  const float wm = warp_max_f32(lm);
  if (wm > a.cur_max) {
    acc_rebase(a, wm);
    uint32_t first = 0xffffffffu;
    if (lm == wm) {
#pragma unroll
      for (int j = UNROLL - 1; j >= 0; --j)
#pragma unroll
        for (int c = 3; c >= 0; --c)
          if (x[j][c] == wm) first = (uint32_t)(seg0 + j * 32 + lane) * 4u + (uint32_t)c;
    }
    a.best_idx = (int)warp_min_u32(first);
  }
  const float nr = -a.r;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    acc_add(x[j][0], nr, a.S0, a.u0);
    acc_add(x[j][1], nr, a.S1, a.u1);
    acc_add(x[j][2], nr, a.S0, a.u0);
    acc_add(x[j][3], nr, a.S1, a.u1);
  }
}


// Loads UNROLL segments, 32 segments apart, starting at p (a lane's pointer into a full slice).
template <int UNROLL>
__device__ __forceinline__ void load_full_slice(uint32_t (&w)[UNROLL][4], const uint4* __restrict__ p) {
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const uint4 q = ld_stream(p + j * 32);  // constant offsets: one pointer per slice
    w[j][0] = q.x; w[j][1] = q.y; w[j][2] = q.z; w[j][3] = q.w;
  }
}
// The same for a slice that runs past seg_end: segments at or past seg_end read as -inf.
template <int UNROLL>
__device__ __forceinline__ void load_ragged_slice(uint32_t (&w)[UNROLL][4], const uint4* __restrict__ row, int seg0,
                                                  int seg_end, int lane, uint32_t fill) {
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const int s = seg0 + j * 32 + lane;
    uint4 q = make_uint4(fill, fill, fill, fill);
    if (s < seg_end) q = ld_stream(row + s);
    w[j][0] = q.x; w[j][1] = q.y; w[j][2] = q.z; w[j][3] = q.w;
  }
}

template <typename T, int UNROLL>
__device__ __forceinline__ void fold_slice(WarpAcc& a, uint32_t (&w)[UNROLL][4], int seg0, int lane) {
  if constexpr (sizeof(T) == 2) {
    fold_slice_bf16<UNROLL>(a, w, seg0, lane);
  } else {
    float x[UNROLL][4];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) x[j][c] = __uint_as_float(w[j][c]);
    fold_slice_f32<UNROLL>(a, x, seg0, lane);
  }
}

// Element-wise slice for rows without 16-byte structure and for the ragged
// tail of a vector row: UNROLL*32 consecutive elements starting at e0.
template <typename T, int UNROLL>
__device__ __forceinline__ void warp_slice_scalar(WarpAcc& a, const T* __restrict__ row, int e0, int e_end,
                                                  int lane) {
  float x[UNROLL];
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    const int e = e0 + j * 32 + lane;
    float v = -INFINITY;
    if (e < e_end) v = (float)row[e];
    x[j] = max_nan_f32(v, kMaskFloor);
  }
  float lm = kMaskFloor;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) lm = fmaxf(lm, x[j]);
  const float wm = warp_max_f32(lm);
  if (wm > a.cur_max) {
    acc_rebase(a, wm);
    uint32_t first = 0xffffffffu;
    if (lm == wm) {
#pragma unroll
      for (int j = UNROLL - 1; j >= 0; --j)
        if (x[j] == wm) first = (uint32_t)(e0 + j * 32 + lane);
    }
    a.best_idx = (int)warp_min_u32(first);
  }
  const float nr = -a.r;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    // out-of-range lanes hold the floor: 2^(floor*log2e - r) = 0 unless the whole
    // piece is masked, in which case the piece vanishes when merged
    acc_add(x[j], nr, a.S0, a.u0);
  }
}

// Lanes -> warp -> block, then one Partial per unit.
__device__ __forceinline__ void block_finish(const WarpAcc& a, Partial* __restrict__ out, int lane, int warp) {
  __shared__ Partial sm[kReduceWarps];
  float S = a.S0 + a.S1, u = a.u0 + a.u1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    S += __shfl_xor_sync(0xffffffffu, S, o);
    u += __shfl_xor_sync(0xffffffffu, u, o);
  }
  if (lane == 0) {
    Partial p;
    p.mx = a.cur_max; p.S = S; p.u = u; p.idx = a.best_idx;
    sm[warp] = p;
  }
  __syncthreads();
  if (warp == 0) {
    Partial p = lane < kReduceWarps ? sm[lane] : empty_partial();
#pragma unroll
    for (int o = kReduceWarps / 2; o > 0; o >>= 1) {
      Partial q = shfl_xor_partial(p, o);
      merge_partial(p, q);
    }
    if (lane == 0) *out = p;
  }
}

// Fused tail: the block that completes a sequence's last unit verifies the
// sequence.  Called by every thread after block_finish; only warp 0 acts.
__device__ __forceinline__ void sequence_tail(const ScanParams& p, int row, int lane, int warp) {
  __shared__ int sm_y[kMaxRows];
  if (warp != 0 || p.tickets == nullptr) return;
  const int K1 = p.K + 1;
  const int b = row / K1;
  unsigned last = 0;
  if (lane == 0) {
    __threadfence();  // the partial written above is visible before the ticket is taken
    const unsigned t = atomicAdd(p.tickets + b, 1u);
    last = (t == (unsigned)(K1 * p.splits) - 1u);
    if (last) {
      p.tickets[b] = 0;  // ready for the next launch
      __threadfence();
    }
  }
  last = __shfl_sync(0xffffffffu, last, 0);
  if (last) {
    __threadfence();  // every lane reads the other blocks' partials after the ticket was seen
    scan_one_sequence(p, b, lane, sm_y);
  }
}

// grid.x = rows * splits.  Vector path.
//   segs_per_split  whole segments per unit (the last unit of a row may be short)
//   nseg            whole segments in a row; elements [nseg*kElems, V) are the ragged tail
template <typename T, int UNROLL>
__global__ void __launch_bounds__(kReduceThreads)
reduce_rows_vec(const T* __restrict__ logits, int64_t row_stride, int V, int nseg, int splits, int segs_per_split,
                Partial* __restrict__ partials, const __grid_constant__ ScanParams tail) {
  constexpr int kE = Seg<T>::kElems;
  const int unit = blockIdx.x;
  const int row = unit / splits, split = unit - row * splits;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* rp = logits + (int64_t)row * row_stride;
  const uint4* rv = reinterpret_cast<const uint4*>(rp);
  const int seg_begin = split * segs_per_split;
  const int seg_end = min(nseg, seg_begin + segs_per_split);

  // Let a programmatic dependent (the stand-alone scan kernel, or the next
  // step's reduction) get scheduled; it waits for this grid's completion before
  // it touches anything this grid writes.
  asm volatile("griddepcontrol.launch_dependents;");

  WarpAcc a;
  acc_init(a);
  constexpr int kSlice = UNROLL * 32;
  constexpr uint32_t kFill = sizeof(T) == 2 ? kNegInf2 : 0xff800000u;
  constexpr int kStride = kReduceWarps * kSlice;
  int s0 = seg_begin + warp * kSlice;
  const uint4* ptr = rv + s0 + lane;
  for (; s0 + kSlice <= seg_end; s0 += kStride, ptr += kStride) {  // full slices: no predicates
    uint32_t w[UNROLL][4];
    load_full_slice<UNROLL>(w, ptr);
    fold_slice<T, UNROLL>(a, w, s0, lane);
  }
  if (s0 < seg_end) {  // at most one slice of a warp runs past the end of the piece
    uint32_t w[UNROLL][4];
    load_ragged_slice<UNROLL>(w, rv, s0, seg_end, lane, kFill);
    fold_slice<T, UNROLL>(a, w, s0, lane);
  }
  // ragged tail (fewer than kElems logits): last unit of the row, last warp
  if (split == splits - 1 && warp == kReduceWarps - 1 && nseg * kE < V)
    warp_slice_scalar<T, 1>(a, rp, nseg * kE, V, lane);
  // Everything above only reads the logits.  When this grid was launched as a
  // programmatic dependent of the previous kernel in the stream, wait for that
  // kernel to complete before the first write (scratch and outputs are shared
  // between consecutive steps).  Otherwise this returns at once.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  block_finish(a, partials + unit, lane, warp);
  sequence_tail(tail, row, lane, warp);
}

// grid.x = rows * splits.  Any alignment, any V.
template <typename T, int UNROLL>
__global__ void __launch_bounds__(kReduceThreads)
reduce_rows_scalar(const T* __restrict__ logits, int64_t row_stride, int V, int splits, int elems_per_split,
                   Partial* __restrict__ partials, const __grid_constant__ ScanParams tail) {
  const int unit = blockIdx.x;
  const int row = unit / splits, split = unit - row * splits;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const T* rp = logits + (int64_t)row * row_stride;
  const int e_begin = split * elems_per_split;
  const int e_end = min(V, e_begin + elems_per_split);
  asm volatile("griddepcontrol.launch_dependents;");
  WarpAcc a;
  acc_init(a);
  constexpr int kSlice = UNROLL * 32;
  for (int e0 = e_begin + warp * kSlice; e0 < e_end; e0 += kReduceWarps * kSlice)
    warp_slice_scalar<T, UNROLL>(a, rp, e0, e_end, lane);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  block_finish(a, partials + unit, lane, warp);
  sequence_tail(tail, row, lane, warp);
}

}  // namespace fly

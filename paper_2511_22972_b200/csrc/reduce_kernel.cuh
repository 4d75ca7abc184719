// Row reduction of the FLy verification step: one streaming pass over the logits
// yields, per row, the running maximum, the softmax normaliser, the weighted sum
// that gives the entropy (Eq. 5) and the greedy token (Eq. 1).
//
// Work decomposition ("flat partition").  The rows of one step are laid end to
// end; a row holds `n` units (a unit is one 16-byte segment on the vector path,
// one logit on the element-wise path).  The grid has G thread blocks, all
// resident at once, and block b reduces the flat unit range [b*Q, (b+1)*Q): the
// same number of bytes for every block, so that they finish together whatever
// the number of rows is.  Where the range crosses a row boundary the block closes
// the row's piece (one 16-byte Partial) and starts the next row.  In the flat
// index space a row spans `span` >= n units (units past n do not exist): span = n
// packs the rows densely (large steps: a block takes a long range, the odd row
// boundary inside it costs little); span = s*Q cuts every row into exactly s
// pieces that never cross a row (small steps, where a boundary inside a block
// would lengthen its critical path by a whole slice).  Row r is covered by the
// blocks (r*span)/Q .. ((r+1)*span-1)/Q, and piece k of a row is stored at
// partials[row * slots + k].
//
// Memory pipeline (vector path).  Every warp owns a small ring in shared memory
// that it fills with asynchronous 16-byte copies (cp.async): kDepth slices of
// UNROLL*32 segments (2 KB each) are in flight per warp while it folds the oldest
// one, 4 blocks x 8 warps per SM (128 KB in flight per SM, none of it in
// registers).  A lane reads back exactly the bytes it copied, so the ring needs
// no barrier.  The whole grid issues its first 2 x 2 KB per warp at once, and a
// block that goes on into the next row starts that row's first slices before it
// merges the finished piece: a grid that runs alone (one step of a decode loop)
// has no second wave and no idle round trip at a row boundary.
//
// Arithmetic.  A warp keeps ONE reference exponent (its running maximum), so a
// slice costs one warp-wide max (redux.sync) and the rescale / index search only
// runs when the maximum actually moves (a handful of times per row).  Per pair of
// logits the steady state is: widen (2), one packed FMA into the base-2
// exponents, two MUFU ex2, one packed add and one packed FMA into the sums
// (fma/add.f32x2: two fp32 operations per issue slot).
#pragma once
#include "fly_common.cuh"
#include "scan_kernel.cuh"

namespace fly {

constexpr int kReduceThreads = 256;
constexpr int kReduceWarps = kReduceThreads / 32;
constexpr int kReduceBlocksPerSM = 4;  // __launch_bounds__ below: <= 64 registers; measured against 3, 5 and 6
constexpr int kDepth = 2;              // slices in flight per warp (3 and 4 measured: no faster)
constexpr int kMaxPend = 8;            // finished pieces a block holds back before it writes them out

// ---- packed fp32 pairs ------------------------------------------------------------------------
using f2 = unsigned long long;  // two fp32 values in one 64-bit register: {lo, hi}

__device__ __forceinline__ f2 pack2(float lo, float hi) {
  f2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) {
  f2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f2 add2(f2 a, f2 b) {
  f2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f2 mul2(f2 a, f2 b) {
  f2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Per-warp streaming state.  S2/u2 are per-lane pairs of accumulators, everything else is warp-uniform.
struct WarpAcc {
  float cur_max;  // raw running maximum (warp-uniform)
  float r;        // cur_max * scale: reference exponent of S and u
  float scale;    // log2(e) / temperature: logit -> base-2 exponent
  int best_idx;   // lowest index holding cur_max (warp-uniform)
  f2 S2, u2;
};

__device__ __forceinline__ void acc_init(WarpAcc& a, float scale) {
  a.cur_max = kMaskFloor;
  a.scale = scale;
  a.r = kMaskFloor * scale;
  a.best_idx = kIdxNone;
  a.S2 = pack2(0.f, 0.f);
  a.u2 = pack2(0.f, 0.f);
}

// Moves the reference exponent to a larger maximum (warp-uniform call).
__device__ __forceinline__ void acc_rebase(WarpAcc& a, float new_max) {
  const float nr = new_max * a.scale;
  const float d = a.r - nr;  // < 0, finite
  const float sc = ex2_approx(d);
  const f2 d2 = pack2(d, d), sc2 = pack2(sc, sc);
  a.u2 = mul2(sc2, fma2(d2, a.S2, a.u2));
  a.S2 = mul2(a.S2, sc2);
  a.r = nr;
  a.cur_max = new_max;
}

// Adds the pair of logits (x0, x1): t = x * scale - r, S += 2^t, u += 2^t * t.
__device__ __forceinline__ void acc_add2(WarpAcc& a, float x0, float x1, f2 sc2, f2 nr2) {
  const f2 t2 = fma2(pack2(x0, x1), sc2, nr2);
  float t0, t1;
  unpack2(t2, t0, t1);
  const f2 e2 = pack2(ex2_approx(t0), ex2_approx(t1));
  a.S2 = add2(a.S2, e2);
  a.u2 = fma2(e2, t2, a.u2);
}

// ---------------------------------------------------------------------------
// Vector path: rows whose base, stride and length are multiples of 16 bytes.
// A "segment" is one 16-byte load: 8 bf16 or 4 fp32 logits.
// ---------------------------------------------------------------------------

template <typename T> struct Seg;
template <> struct Seg<__nv_bfloat16> { static constexpr int kElems = 8; };
template <> struct Seg<float> { static constexpr int kElems = 4; };

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

__device__ __forceinline__ uint32_t smem_addr_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Asynchronous 16-byte copy global -> shared (bypasses L1, no register staging).
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global.L2::128B [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// First half of folding a slice of bf16 logits (w[j] = segment seg0 + j*32 + lane of the row, 8 logits;
// segments at or past seg_end do not belong to the piece): masks and clamps the data and returns the
// lane's maximum.  Masked entries are clamped to the floor (NaN survives the clamp and ends in S).
template <int UNROLL>
__device__ __forceinline__ float slice_max_bf16(uint32_t (&w)[UNROLL][4], int seg0, int seg_end, int lane) {
  constexpr uint32_t kFloor2 = 0xc974c974u;  // bf16(kMaskFloor) twice
  if (seg0 + UNROLL * 32 > seg_end) {        // ragged slice (warp-uniform)
#pragma unroll
    for (int j = 0; j < UNROLL; ++j)
      if (seg0 + j * 32 + lane >= seg_end) w[j][0] = w[j][1] = w[j][2] = w[j][3] = kNegInf2;
  }
  uint32_t lm2 = kFloor2;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      w[j][c] = bf2_max_nan(w[j][c], kFloor2);
      lm2 = bf2_max(lm2, w[j][c]);
    }
  return fmaxf(bf16lo(lm2), bf16hi(lm2));
}

// Second half: warp maximum, rebase when it moved, then the exponentials.
template <int UNROLL>
__device__ __forceinline__ void slice_sum_bf16(WarpAcc& a, const uint32_t (&w)[UNROLL][4], float lm, int seg0, int lane) {
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
  const f2 nr2 = pack2(-a.r, -a.r), sc2 = pack2(a.scale, a.scale);
#pragma unroll
  for (int j = 0; j < UNROLL; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc_add2(a, bf16lo(w[j][c]), bf16hi(w[j][c]), sc2, nr2);
}

// The same two halves for fp32 logits: w[j] holds 4 logits as raw bits.
template <int UNROLL>
__device__ __forceinline__ float slice_max_f32(uint32_t (&w)[UNROLL][4], int seg0, int seg_end, int lane) {
  if (seg0 + UNROLL * 32 > seg_end) {
#pragma unroll
    for (int j = 0; j < UNROLL; ++j)
      if (seg0 + j * 32 + lane >= seg_end) w[j][0] = w[j][1] = w[j][2] = w[j][3] = 0xff800000u;
  }
  float lm = kMaskFloor;
#pragma unroll
  for (int j = 0; j < UNROLL; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float x = max_nan_f32(__uint_as_float(w[j][c]), kMaskFloor);
      w[j][c] = __float_as_uint(x);
      lm = fmaxf(lm, x);
    }
  return lm;
}
template <int UNROLL>
__device__ __forceinline__ void slice_sum_f32(WarpAcc& a, const uint32_t (&w)[UNROLL][4], float lm, int seg0, int lane) {
  const float wm = warp_max_f32(lm);
  if (wm > a.cur_max) {
    acc_rebase(a, wm);
    uint32_t first = 0xffffffffu;
    if (lm == wm) {
#pragma unroll
      for (int j = UNROLL - 1; j >= 0; --j)
#pragma unroll
        for (int c = 3; c >= 0; --c)
          if (__uint_as_float(w[j][c]) == wm) first = (uint32_t)(seg0 + j * 32 + lane) * 4u + (uint32_t)c;
    }
    a.best_idx = (int)warp_min_u32(first);
  }
  const f2 nr2 = pack2(-a.r, -a.r), sc2 = pack2(a.scale, a.scale);
#pragma unroll
  for (int j = 0; j < UNROLL; ++j) {
    acc_add2(a, __uint_as_float(w[j][0]), __uint_as_float(w[j][1]), sc2, nr2);
    acc_add2(a, __uint_as_float(w[j][2]), __uint_as_float(w[j][3]), sc2, nr2);
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
  const f2 nr2 = pack2(-a.r, -a.r), sc2 = pack2(a.scale, a.scale);
  // out-of-range lanes hold the floor: 2^(floor*scale - r) = 0 unless the whole
  // piece is masked, in which case the piece vanishes when merged
  if constexpr (UNROLL == 1) {
    acc_add2(a, x[0], kMaskFloor, sc2, nr2);
  } else {
#pragma unroll
    for (int j = 0; j < UNROLL; j += 2) acc_add2(a, x[j], x[j + 1], sc2, nr2);
  }
}

// One piece on the element-wise path: logits [e_begin, e_end) of the row.
template <typename T, int UNROLL>
__device__ __forceinline__ void reduce_piece_scalar(WarpAcc& a, const T* __restrict__ rp, int e_begin, int e_end, int lane,
                                                    int warp) {
  constexpr int kSlice = UNROLL * 32;
  for (int e0 = e_begin + warp * kSlice; e0 < e_end; e0 += kReduceWarps * kSlice)
    warp_slice_scalar<T, UNROLL>(a, rp, e0, e_end, lane);
}

// Geometry of one launch (see the head of this file).
struct ReducePlan {
  int64_t n;       // units per row
  int64_t span;    // units a row takes in the flat index space (>= n)
  int64_t Q;       // units per block
  int64_t total;   // rows * span
  int pieces;      // > 0: span = pieces * Q, block b is piece b % pieces of row b / pieces (32-bit arithmetic)
  int slots;       // Partial slots per row (>= the largest number of pieces of any row)
  int V;
  int64_t row_stride;  // elements
  float scale;     // log2(e) / temperature
  int wait_first;  // 1: wait for the previous kernel in the stream before the first read (plain stream
                   //    order); 0: the logits are known to be complete, wait only before the first write
};

// Lanes -> warp -> block; warp 0 / lane 0 ends up with the piece's Partial.  sm: kReduceWarps Partials of
// shared memory; consecutive pieces of a block alternate between two such buffers, so one barrier per
// piece is enough.
__device__ __forceinline__ Partial block_finish(const WarpAcc& a, Partial* sm, int lane, int warp) {
  float S0, S1, u0, u1;
  unpack2(a.S2, S0, S1);
  unpack2(a.u2, u0, u1);
  float S = S0 + S1, u = u0 + u1;
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
  Partial p = empty_partial();
  if (warp == 0) {
    if (lane < kReduceWarps) p = sm[lane];
#pragma unroll
    for (int o = kReduceWarps / 2; o > 0; o >>= 1) {
      Partial q = shfl_xor_partial(p, o);
      merge_partial(p, q, a.scale);
    }
  }
  return p;
}

// A finished piece that has not been written out yet.
struct __align__(16) Pending {
  Partial p;
  int row, slot;
  unsigned units;
  int pad;
};

// Fused tail: the block that completes a sequence verifies it.  A sequence's arrival counter counts the
// units (segments or logits) of its K+1 rows that have been reduced; the block whose piece brings it to
// (K+1) * n has seen every other piece's ticket, hence (after the fences) every other Partial.  Called by
// warp 0 once the piece's Partial is in global memory.
__device__ __forceinline__ void sequence_tail(const ScanParams& p, int row, unsigned units, int lane, int* sm_y) {
  const int K1 = p.K + 1;
  const int b = row / K1;
  unsigned last = 0;
  if (lane == 0) {
    const unsigned t = atomicAdd(p.tickets + b, units);
    last = (t + units == (unsigned)K1 * (unsigned)p.units_per_row);
  }
  last = __shfl_sync(0xffffffffu, last, 0);
  if (last) {
    __threadfence();  // every lane reads the other blocks' partials after the ticket was seen
    scan_one_sequence(p, b, lane, sm_y);
    if (lane == 0) p.tickets[b] = 0;  // ready for the next launch (ordered by the end of this kernel; off the critical path)
  }
}

// Writes the held-back pieces out and takes their tickets (warp 0).
__device__ __forceinline__ void flush_pending(const Pending* pend, int np, int slots, Partial* __restrict__ partials,
                                              const ScanParams& tail, int lane, int* sm_y) {
  if (lane < np) partials[(int64_t)pend[lane].row * slots + pend[lane].slot] = pend[lane].p;
  if (tail.tickets == nullptr) return;
  __threadfence();  // the partials written above are visible ...
  if (np > 1) {     // (one piece: lane 0 wrote it and lane 0 takes its ticket, its own fence is enough)
    __syncwarp();
    __threadfence();  // ... before lane 0 takes any ticket
  }
  for (int k = 0; k < np; ++k) sequence_tail(tail, pend[k].row, pend[k].units, lane, sm_y);
}

// grid.x = ceil(total / Q).  VEC: rows are 16-byte structured (a unit is a segment); else any alignment, any V.
template <typename T, int UNROLL, bool VEC>
__global__ void __launch_bounds__(kReduceThreads, kReduceBlocksPerSM)
reduce_rows_flat(const T* __restrict__ logits, const __grid_constant__ ReducePlan g, Partial* __restrict__ partials,
                 const __grid_constant__ ScanParams tail) {
  constexpr int kE = Seg<T>::kElems;
  constexpr int kSlice = UNROLL * 32;
  constexpr int kStride = kReduceWarps * kSlice;
  extern __shared__ __align__(16) uint4 ring[];  // VEC: kReduceWarps * kDepth * kSlice segments
  __shared__ Partial sm_part[2][kReduceWarps];
  __shared__ Pending pend[kMaxPend];
  __shared__ int sm_y[kMaxRows];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // The grid is launched as a programmatic dependent of the previous kernel in the stream.  Plain
  // stream order: wait for that kernel to complete (and its writes to be visible) before anything is
  // read.  With inputs_ready the reads start at once and the wait comes before the first write.
  bool waited = g.wait_first != 0;
  if (waited) asm volatile("griddepcontrol.wait;" ::: "memory");
  // Let the next kernel in the stream get scheduled early if it asks for that; it waits for this
  // grid's completion before it touches anything this grid writes.
  asm volatile("griddepcontrol.launch_dependents;");

  int row, u0, u1, slot;  // the current piece: units [u0, u1) of `row`, stored in the row's slot `slot`
  int64_t left, take;     // flat units of this block not yet assigned to a piece; flat units the current piece takes
  if (g.pieces > 0) {     // whole pieces of rows: one per block, 32-bit arithmetic (the common small-step case)
    row = (int)blockIdx.x / g.pieces;
    slot = (int)blockIdx.x - row * g.pieces;
    u0 = slot * (int)g.Q;
    u1 = min((int)g.n, u0 + (int)g.Q);
    left = take = g.Q;
  } else {
    const int64_t f0 = (int64_t)blockIdx.x * g.Q;
    const int64_t f_end = min(f0 + g.Q, g.total);
    row = (int)(f0 / g.span);
    u0 = (int)(f0 - (int64_t)row * g.span);
    slot = (int)((int64_t)blockIdx.x - ((int64_t)row * g.span) / g.Q);     // pieces of the row that earlier blocks hold
    u1 = (int)min(g.n, (int64_t)u0 + (f_end - f0));
    left = f_end - f0;                                                     // (a row ends at its span, not at n)
    take = min((int64_t)g.span - u0, left);
  }

  // Copy side of the pipeline.  A warp's slices of the piece [pu0, pu1) of the row at `prow` start at
  // ps = pu0 + warp * kSlice and lie kStride apart; issue() copies the next one into a ring stage.
  const uint32_t ring_warp = smem_addr_u32(ring) + (uint32_t)((warp * kDepth * kSlice + lane) * 16);
  const uint4* psrc = nullptr;
  int ps = 0, pend_seg = 0;
  auto open_piece = [&](int prow, int pu0, int pu1) {
    psrc = reinterpret_cast<const uint4*>(logits + (int64_t)prow * g.row_stride) + lane;
    ps = pu0 + warp * kSlice;
    pend_seg = pu1;
  };
  auto issue = [&](int stage) {
    if (ps < pend_seg) {
      const uint32_t dst = ring_warp + (uint32_t)(stage * kSlice * 16);
      if (ps + kSlice <= pend_seg) {
#pragma unroll
        for (int j = 0; j < UNROLL; ++j) cp_async16(dst + j * 512, psrc + ps + j * 32);
      } else {
#pragma unroll
        for (int j = 0; j < UNROLL; ++j)
          if (ps + j * 32 + lane < pend_seg) cp_async16(dst + j * 512, psrc + ps + j * 32);
      }
      ps += kStride;
    }
    cp_async_commit();  // one group per call, empty or not: the folding side counts groups
  };
  if constexpr (VEC) {
    open_piece(row, u0, u1);
#pragma unroll
    for (int d = 0; d < kDepth; ++d) issue(d);
  }

  // The acceptance scan at the end of the step reads draft tokens and carried state, which nothing has
  // touched yet: pull them into L2 now so that the last block does not wait on DRAM for them.
  if (tail.tickets != nullptr && (int)blockIdx.x < tail.B && warp == 1) {
    const int32_t* d = tail.draft + (int64_t)blockIdx.x * tail.K;
    if (lane * 32 < tail.K) asm volatile("prefetch.global.L2 [%0];" ::"l"(d + lane * 32));
    if (lane == 31 && tail.state_in) asm volatile("prefetch.global.L2 [%0];" ::"l"(tail.state_in + (int64_t)blockIdx.x * 3));
  }

  int parity = 0, np = 0;
  while (true) {
    const T* rp = logits + (int64_t)row * g.row_stride;
    WarpAcc a;
    acc_init(a, g.scale);
    left -= take;
    if constexpr (VEC) {
      int stage = 0;
      for (int s0 = u0 + warp * kSlice; s0 < u1; s0 += kStride) {
        cp_async_wait<kDepth - 1>();  // the oldest slice in flight has landed
        uint32_t w[UNROLL][4];
        const uint4* src = ring + (warp * kDepth + stage) * kSlice + lane;
#pragma unroll
        for (int j = 0; j < UNROLL; ++j) {
          const uint4 q = src[j * 32];
          w[j][0] = q.x; w[j][1] = q.y; w[j][2] = q.z; w[j][3] = q.w;
        }
        float lm;
        if constexpr (sizeof(T) == 2) lm = slice_max_bf16<UNROLL>(w, s0, u1, lane);
        else lm = slice_max_f32<UNROLL>(w, s0, u1, lane);
        // every register of the slice has been consumed once, so the stage's bytes are out of shared
        // memory: refill it with the slice kDepth ahead
        issue(stage);
        if constexpr (sizeof(T) == 2) slice_sum_bf16<UNROLL>(a, w, lm, s0, lane);
        else slice_sum_f32<UNROLL>(a, w, lm, s0, lane);
        stage = stage + 1 == kDepth ? 0 : stage + 1;
      }
      // This warp's ring is empty now.  If the block goes on into the next row, start that piece's first
      // slices before the block-wide merge below, so that the row boundary costs no memory round trip.
      if (left > 0) {
        cp_async_wait<0>();
        open_piece(row + 1, 0, (int)min(g.n, left));
#pragma unroll
        for (int d = 0; d < kDepth; ++d) issue(d);
      }
      // ragged tail (fewer than kElems logits): the piece that ends the row, last warp
      if (u1 == (int)g.n && warp == kReduceWarps - 1 && (int)g.n * kE < g.V) warp_slice_scalar<T, 1>(a, rp, (int)g.n * kE, g.V, lane);
    } else {
      reduce_piece_scalar<T, UNROLL>(a, rp, u0, u1, lane, warp);
    }
    const Partial p = block_finish(a, sm_part[parity], lane, warp);
    if (warp == 0 && lane == 0) {
      Pending q;
      q.p = p; q.row = row; q.slot = slot; q.units = (unsigned)(u1 - u0); q.pad = 0;
      pend[np] = q;
    }
    ++np;
    parity ^= 1;
    const bool done = left <= 0;
    if (np == kMaxPend || done) {
      // Everything so far only read the logits.  Scratch and outputs are shared with the previous step:
      // with inputs_ready its kernel may still be running, so wait for it before the first write.
      if (!waited) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
      }
      if (warp == 0) {
        __syncwarp();
        flush_pending(pend, np, g.slots, partials, tail, lane, sm_y);
        __syncwarp();
      }
      np = 0;
    }
    if (done) break;
    ++row;
    u0 = 0;
    u1 = (int)min(g.n, left);
    take = min((int64_t)g.span, left);
    slot = 0;
  }
  if constexpr (VEC) cp_async_wait<0>();
}

}  // namespace fly

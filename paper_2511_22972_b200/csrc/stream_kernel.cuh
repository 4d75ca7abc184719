// Row reduction of the FLy verification step as a persistent streaming kernel:
// the same per-logit arithmetic as reduce_kernel.cuh (Eq. 1, Eq. 5), with the
// logits staged through a shared-memory ring by bulk asynchronous copies.
//
// Why a second form.  With one thread block per (row, piece) the bytes in
// flight are tied to the registers of resident warps and every block pays a
// pipeline fill and drain; a grid that runs alone reaches ~58 % of the DRAM
// bandwidth.  Here one CTA per SM walks a contiguous range of units
// (unit = (row, piece)); a producer thread keeps kStages bulk copies of
// kChunkBytes in flight whatever the consumers are doing, and runs ahead across
// unit boundaries, so the memory pipe never drains between units.
//
// Roles: warps 0..15 consume (each folds a 1 KB slice of every chunk: two
// 16-byte segments per lane), warp 16 lane 0 produces.  full[s] is completed by
// the copy's byte count, empty[s] by one arrival per consumer warp.  At the end
// of a unit the consumer warps merge their states (named barrier, double
// buffered), warp 0 writes the unit's Partial and takes the sequence's ticket;
// the CTA that completes a sequence runs the acceptance scan for it.
//
// Every barrier wait is bounded.  A wait that runs out marks the CTA dead: its
// warps keep walking the loop (so that named barriers still match) but skip all
// work, and the status word tells the host.
#pragma once
#include "fly_common.cuh"
#include "mbarrier.cuh"
#include "reduce_kernel.cuh"
#include "scan_kernel.cuh"

namespace fly {
namespace stream {

constexpr int kConsumerWarps = 16;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kSegsPerLane = 2;                                    // 16-byte segments per lane and chunk
constexpr int kChunkSegs = kConsumerWarps * 32 * kSegsPerLane;     // 1024 segments
constexpr int kChunkBytes = kChunkSegs * 16;                       // 16 KB
constexpr int kStages = 6;
constexpr int kRingBytes = kStages * kChunkBytes;                  // 96 KB: two CTAs (consecutive grids) fit on an SM
constexpr int kSmemBytes = kRingBytes + 2 * kStages * 8 + 2 * kConsumerWarps * 16 + 16 + 128;
constexpr int kErrTimeoutStream = 4;

struct Params {
  const void* logits;
  int64_t row_stride;   // elements
  int V;
  int nseg;             // whole 16-byte segments in a row
  int splits;           // pieces per row
  int segs_per_split;
  int units;            // rows * splits
  Partial* partials;    // [units]
  int* status;
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 512;" ::: "memory"); }

template <typename T>
__global__ void __launch_bounds__(kThreads, 2)
reduce_rows_stream(const Params p, const __grid_constant__ ScanParams tail) {
  constexpr int kE = Seg<T>::kElems;
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t ring = smem_u32(smem);
  const uint32_t bar0 = ring + kRingBytes;
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto empty = [&](int s) { return bar0 + 8u * (kStages + s); };
  Partial* merge_buf = reinterpret_cast<Partial*>(smem + kRingBytes + 2 * kStages * 8);  // [2][kConsumerWarps]
  volatile int* dead = reinterpret_cast<volatile int*>(smem + kRingBytes + 2 * kStages * 8 + 2 * kConsumerWarps * 16);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), kConsumerWarps); }
    *dead = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // Let the next grid in the stream start: it only reads its logits until its own
  // griddepcontrol.wait, which it executes before its first write.
  asm volatile("griddepcontrol.launch_dependents;");

  // contiguous range of units of this CTA
  const int u0 = (int)(((int64_t)p.units * blockIdx.x) / gridDim.x);
  const int u1 = (int)(((int64_t)p.units * (blockIdx.x + 1)) / gridDim.x);
  const T* base = static_cast<const T*>(p.logits);

  if (warp == kConsumerWarps) {
    // ---------------- producer ----------------
    if (lane == 0) {
      int n = 0;
      for (int u = u0; u < u1 && !*dead; ++u) {
        const int row = u / p.splits, split = u - row * p.splits;
        const int seg_begin = split * p.segs_per_split;
        const int seg_end = min(p.nseg, seg_begin + p.segs_per_split);
        const uint8_t* src = reinterpret_cast<const uint8_t*>(base + (int64_t)row * p.row_stride) + (int64_t)seg_begin * 16;
        for (int s0 = seg_begin; s0 < seg_end; s0 += kChunkSegs, ++n) {
          const int st = n % kStages;
          if (!mbar_wait(empty(st), ((n / kStages) & 1) ^ 1, p.status, kErrTimeoutStream)) { *dead = 1; break; }
          const uint32_t bytes = (uint32_t)min(kChunkSegs, seg_end - s0) * 16u;
          mbar_expect_tx(full(st), bytes);
          bulk_load(ring + st * kChunkBytes, src + (int64_t)(s0 - seg_begin) * 16, bytes, full(st));
        }
      }
    }
  } else {
    // ---------------- consumers ----------------
    int n = 0;
    for (int u = u0; u < u1; ++u) {
      const int row = u / p.splits, split = u - row * p.splits;
      const int seg_begin = split * p.segs_per_split;
      const int seg_end = min(p.nseg, seg_begin + p.segs_per_split);
      WarpAcc a;
      acc_init(a);
      for (int s0 = seg_begin; s0 < seg_end; s0 += kChunkSegs, ++n) {
        const int st = n % kStages;
        if (!*dead && !mbar_wait(full(st), (n / kStages) & 1, p.status, kErrTimeoutStream)) *dead = 1;
        if (*dead) continue;
        const int seg0 = s0 + warp * (32 * kSegsPerLane);  // first segment of this warp's slice, within the row
        const uint32_t src = ring + st * kChunkBytes + (uint32_t)(warp * (32 * kSegsPerLane) + lane) * 16u;
        if constexpr (sizeof(T) == 2) {
          uint32_t w[kSegsPerLane][4];
#pragma unroll
          for (int j = 0; j < kSegsPerLane; ++j) {
            uint4 q = make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);
            if (seg0 + j * 32 + lane < seg_end) q = lds128(src + j * 512);
            w[j][0] = q.x; w[j][1] = q.y; w[j][2] = q.z; w[j][3] = q.w;
          }
          fold_slice_bf16<kSegsPerLane>(a, w, seg0, lane);
          __syncwarp();
          if (lane == 0) mbar_arrive(empty(st));  // every lane has consumed its part: the stage may be refilled
        } else {
          float x[kSegsPerLane][4];
#pragma unroll
          for (int j = 0; j < kSegsPerLane; ++j) {
            uint4 q = make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
            if (seg0 + j * 32 + lane < seg_end) q = lds128(src + j * 512);
            x[j][0] = __uint_as_float(q.x); x[j][1] = __uint_as_float(q.y);
            x[j][2] = __uint_as_float(q.z); x[j][3] = __uint_as_float(q.w);
          }
          fold_slice_f32<kSegsPerLane>(a, x, seg0, lane);
          __syncwarp();
          if (lane == 0) mbar_arrive(empty(st));
        }
      }
      // ragged tail of the row (fewer than kElems logits): last piece, last warp, straight from global memory
      if (!*dead && split == p.splits - 1 && warp == kConsumerWarps - 1 && p.nseg * kE < p.V)
        warp_slice_scalar<T, 1>(a, base + (int64_t)row * p.row_stride, p.nseg * kE, p.V, lane);

      // ---- end of the unit: lanes -> warp -> CTA ----
      float S = a.S0 + a.S1, uu = a.u0 + a.u1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        S += __shfl_xor_sync(0xffffffffu, S, o);
        uu += __shfl_xor_sync(0xffffffffu, uu, o);
      }
      Partial* buf = merge_buf + ((u - u0) & 1) * kConsumerWarps;
      if (lane == 0) {
        Partial q;
        q.mx = a.cur_max; q.S = S; q.u = uu; q.idx = a.best_idx;
        buf[warp] = q;
      }
      consumer_bar();
      if (warp == 0 && !*dead) {
        Partial q = lane < kConsumerWarps ? buf[lane] : empty_partial();
#pragma unroll
        for (int o = kConsumerWarps / 2; o > 0; o >>= 1) {
          const Partial r = shfl_xor_partial(q, o);
          merge_partial(q, r);
        }
        // first write of this CTA: the previous kernel in the stream must have completed
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (lane == 0) p.partials[u] = q;
        sequence_tail(tail, row, lane, 0);
      }
    }
  }
  if (*(volatile int*)p.status != 0) {  // after a failed wait: let copies in flight land before the ring is handed back
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) {}
  }
}

}  // namespace stream
}  // namespace fly

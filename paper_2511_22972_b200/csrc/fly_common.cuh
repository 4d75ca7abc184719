// Shared device-side definitions of the FLy verification kernels (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace fly {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// Logits at or below this are treated as masked: they are clamped to it so that
// every intermediate stays finite (a -inf logit has p = 0 and adds nothing to
// the entropy; 0 * -inf would otherwise poison the weighted sum).  The value is
// exactly representable in bf16 and small enough in magnitude that the rounding
// of floor * log2(e) is negligible; a row whose maximum does not exceed it
// counts as having no finite entry.
constexpr float kMaskFloor = -999424.0f;
constexpr int kIdxNone = 0x7fffffff;

constexpr uint32_t kFlagNonFinite = 1u;
constexpr uint32_t kFlagBadDraft = 2u;
constexpr uint32_t kFlagBadTarget = 4u;
constexpr uint32_t kFlagBadState = 8u;
constexpr uint32_t kFlagStepFailed = 16u;

// Running state of one (piece of a) row in the base-2 domain.
//   mx   largest logit seen (raw value; decides the argmax)
//   S    sum 2^(z - r)            z = logit * scale,  r = mx * scale,  scale = log2(e) / temperature
//   u    sum 2^(z - r) * (z - r)
//   idx  lowest index holding mx
// Entropy in nats (numerator of Eq. 5):  H = ln2 * (log2 S - u / S), for any
// common reference r, so pieces can be rebased and added.
struct __align__(16) Partial {
  float mx;
  float S;
  float u;
  int idx;
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max_nan_f32(float a, float b) {
  float y;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(y) : "f"(a), "f"(b));
  return y;
}
__device__ __forceinline__ float warp_max_f32(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ uint32_t warp_min_u32(uint32_t v) { return __reduce_min_sync(0xffffffffu, v); }

// Rebase identity: sum 2^(z-r')(z-r') = 2^(r-r') * (u + (r-r') S).
// Merges b into a; on equal maxima the lower index wins (Eq. 1 tie rule).
__device__ __forceinline__ void merge_partial(Partial& a, const Partial& b, float scale) {
  const float ra = a.mx * scale, rb = b.mx * scale;
  const float r = fmaxf(ra, rb);
  const float da = ra - r, db = rb - r;  // <= 0, finite (mx is clamped to the mask floor)
  const float ea = ex2_approx(da), eb = ex2_approx(db);
  const float S = a.S * ea + b.S * eb;
  const float u = ea * fmaf(da, a.S, a.u) + eb * fmaf(db, b.S, b.u);
  if (b.mx > a.mx || (b.mx == a.mx && b.idx < a.idx)) a.idx = b.idx;
  a.mx = fmaxf(a.mx, b.mx);
  a.S = S;
  a.u = u;
}

__device__ __forceinline__ Partial empty_partial() {
  Partial p;
  p.mx = kMaskFloor;
  p.S = 0.f;
  p.u = 0.f;
  p.idx = kIdxNone;
  return p;
}

__device__ __forceinline__ Partial shfl_xor_partial(const Partial& p, int lane_mask) {
  Partial q;
  q.mx = __shfl_xor_sync(0xffffffffu, p.mx, lane_mask);
  q.S = __shfl_xor_sync(0xffffffffu, p.S, lane_mask);
  q.u = __shfl_xor_sync(0xffffffffu, p.u, lane_mask);
  q.idx = __shfl_xor_sync(0xffffffffu, p.idx, lane_mask);
  return q;
}

}  // namespace fly

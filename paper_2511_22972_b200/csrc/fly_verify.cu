// Host side of the C ABI declared in include/fly_verify.h: argument checks,
// launch-shape selection and kernel launches.  No torch types, no allocation
// inside fly_verify_run.
#include "fly_verify.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include <cudaTypedefs.h>

#include "fly_common.cuh"
#include "lmhead_kernel.cuh"
#include "pld_kernel.cuh"
#include "reduce_kernel.cuh"
#include "scan_kernel.cuh"

namespace {

constexpr int kMaxSplits = 32;   // Partial slots per row in a handle's scratch
// 16-byte copies per lane and slice in the row-reduction kernel (a warp's ring holds fly::kDepth slices).
constexpr int kReduceUnroll = 4;
constexpr int64_t kMinBlockBytes = 16384;   // a block that gets less than this is all fixed cost
constexpr int kMaxK = 63;

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    want = dev;
  }
  ~DeviceGuard() {
    if (ok && prev != want) cudaSetDevice(prev);
  }
  int want = -1;
};

}  // namespace

struct fly_verify {
  fly_verify_config_t cfg;
  int sm_count = 148;
  int64_t max_rows = 0;
  fly::Partial* partials = nullptr;  // [max_rows * kMaxSplits]
  unsigned int* tickets = nullptr;   // [max_batch], zero between launches
  int forced_splits = 0;
  int scan_mode = 0;   // 0: fused tail, 1: separate kernel
  int last_launches = 0;
  int last_cuda_error = 0;
  // fused LM-head path (cfg.hidden > 0)
  fly::Partial* lm_partials = nullptr;  // [max_rows * sm_count]: one partial state per row and CTA
  fly::Partial* lm_folded = nullptr;    // [max_rows]: partial states folded over CTAs (fused path) or ranks
  int* lm_status = nullptr;             // device word: first bounded wait that ran out (sticky until read)
  int lm_pairs = 0;                     // CTA pairs that can be resident at once
  int weight_vd = 0;                    // 0: weight [hidden, V]; 1: weight [V, hidden]
  PFN_cuTensorMapEncodeTiled encode_tiled = nullptr;
  CUtensorMap map_w, map_h;             // cached for (map_w_ptr, map_h_ptr, map_h_rows)
  const void* map_w_ptr = nullptr;
  const void* map_h_ptr = nullptr;
  int64_t map_h_rows = 0;
  void* st_hidden = nullptr;            // staging of fly_verify_run_host
  size_t st_hidden_bytes = 0;
  // staging for fly_verify_run_host (allocated on first use)
  void* st_logits = nullptr;
  size_t st_logits_bytes = 0;
  int32_t* st_ints = nullptr;  // device: draft | state_in | target tokens || state_out | accept | rollback | tokens | argmax | flags | entropy
  int32_t* st_host = nullptr;  // page-locked host copy of the same block
};

namespace {

fly_status_t cuda_fail(fly_verify* h, cudaError_t e) {
  h->last_cuda_error = (int)e;
  return FLY_ERR_CUDA;
}

// Launch geometry of the row reduction (the flat index space described at the head of reduce_kernel.cuh).
//   n      units per row, min_units: a block should not get less than this
//   cap    Partial slots available per row (>= 1)
struct FlatPlan {
  int64_t Q = 1;      // units per block
  int64_t span = 1;   // units a row takes in the flat index space
  int grid = 1;
  int slots = 1;
  int pieces = 0;     // > 0: every row is cut into exactly this many pieces (span = pieces * Q)
};
// Launch shape.  Measured on the bench workloads (9 .. 2304 rows of 128 - 300 KB): whole pieces of rows, one per
// block, are at least as fast as packed rows whenever they fill the resident slots reasonably well - a row boundary
// inside a block drains that block's copy ring once, and the hardware scheduler back-fills a second wave well.
// A block's warps walk its piece in strides of `stride_units` (one slice per warp), so a piece of 3.1 strides costs
// its slowest warp 4 slices: among the piece counts that fit, the one with the fewest slices on the busiest SM wins.
//   plain stream order   the grid fits on the device at once (4 blocks per SM); cost = blocks on the busiest SM x
//                        slices per warp, ties go to the count nearest two blocks per SM (the next step's blocks
//                        can then already be resident, waiting); more rows than slots: whole rows, several waves
//   inputs_ready         throughput, not latency: few large pieces (a quarter of a block per SM and step is
//                        enough, consecutive steps overlap many deep), the count with the fewest slices per row
//   packed rows          only where whole pieces would leave more than a quarter of the last wave's slots empty
int64_t piece_units(int64_t n, int64_t s) {
  int64_t q = (n + s - 1) / s;
  if (s > 1) q = (q + 7) / 8 * 8;  // pieces start on 128-byte boundaries of the row
  return q;
}
FlatPlan plan_flat(int sm_count, int64_t rows, int64_t n, int64_t min_units, int64_t stride_units, int cap,
                   bool inputs_ready, int forced) {
  FlatPlan pl;
  const int64_t gmax = (int64_t)sm_count * fly::kReduceBlocksPerSM;
  int64_t smax = n / min_units;  // pieces of at least min_units
  if (smax > cap) smax = cap;
  if (smax < 1) smax = 1;
  auto slices = [&](int64_t s) { return (piece_units(n, s) + stride_units - 1) / stride_units; };
  int64_t s = 0;  // > 0: every row is cut into exactly s pieces
  if (cap < 2) {
    s = 1;        // one slot per row: whole rows
  } else if (forced > 0) {
    s = forced < cap ? forced : cap;
  } else if (inputs_ready) {
    int64_t target = sm_count / (4 * rows);
    if (target > smax) target = smax;
    if (target < 1) target = 1;
    int64_t best = -1;
    for (int64_t c = 1; c <= target; ++c) {
      const int64_t cost = c * slices(c);  // slices per row
      if (best < 0 || cost <= best) { best = cost; s = c; }
    }
  } else if (rows >= gmax) {
    s = 1;
  } else {
    int64_t best = -1, best_dist = 0;
    for (int64_t c = 1; c <= smax && rows * c <= gmax; ++c) {
      const int64_t cost = ((rows * c + sm_count - 1) / sm_count) * slices(c);
      int64_t dist = rows * c - 2 * sm_count;
      if (dist < 0) dist = -dist;
      if (best < 0 || cost < best || (cost == best && dist < best_dist)) { best = cost; best_dist = dist; s = c; }
    }
    if (s < 1) s = 1;
  }
  if (s > 0 && cap >= 2 && forced <= 0 && !inputs_ready) {
    int64_t s_fill = gmax / rows;  // the most pieces per row that still fit at once
    if (s_fill > smax) s_fill = smax;
    if (s_fill < 1) s_fill = 1;
    const int64_t blocks = rows * s_fill, waves = (blocks + gmax - 1) / gmax;
    const bool could_fill = rows * n / min_units >= gmax;  // enough work for a full grid at all
    if (could_fill && 4 * blocks < 3 * waves * gmax) {
      // the last wave would be mostly empty: pack the rows end to end and cut the range evenly instead
      s = 0;
      const int64_t Qf = (rows * n + gmax - 1) / gmax;
      pl.Q = (Qf + 63) / 64 * 64;  // piece starts on 1 KB boundaries of the row where the row length allows
      const int64_t qmin = (n + (cap - 1) - 1) / (cap - 1);  // a row never spans more than cap blocks
      if (pl.Q < qmin) pl.Q = qmin;
      pl.span = n;
    }
  }
  if (s > 0) {
    if (s > n) s = n;
    pl.Q = piece_units(n, s);
    s = (n + pl.Q - 1) / pl.Q;                   // pieces that are not empty
    pl.span = s * pl.Q;
    pl.pieces = (int)s;
  }
  const int64_t total = rows * pl.span;
  pl.grid = (int)((total + pl.Q - 1) / pl.Q);
  const int64_t most = s > 0 ? s : (n + pl.Q - 1) / pl.Q + 1;
  pl.slots = (int)(most < cap ? most : cap);
  return pl;
}

void fill_launch(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, unsigned grid, unsigned block, cudaStream_t st,
                 bool programmatic) {
  memset(cfg, 0, sizeof(*cfg));
  cfg->gridDim = dim3(grid);
  cfg->blockDim = dim3(block);
  cfg->dynamicSmemBytes = 0;
  cfg->stream = st;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = programmatic ? 1 : 0;
  cfg->attrs = attr;
  cfg->numAttrs = 1;
}

// Shared memory of the row reduction's cp.async rings (vector path), per block.
constexpr int kReduceRingBytes = fly::kReduceWarps * fly::kDepth * kReduceUnroll * 32 * 16;

// Function attributes are per device: set them once on every device that launches the row reduction.
// The rings of all resident blocks only fit on an SM whose L1/shared split favours shared memory.
constexpr int kMaxDevices = 64;
void ensure_reduce_attrs(int device) {
  static std::mutex mu;
  static bool done[kMaxDevices] = {};
  if (device >= 0 && device < kMaxDevices) {
    std::lock_guard<std::mutex> lock(mu);
    if (done[device]) return;
    done[device] = true;
  }
  auto set = [](auto kernel) {
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kReduceRingBytes);
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  };
  set(fly::reduce_rows_flat<__nv_bfloat16, kReduceUnroll, true>);
  set(fly::reduce_rows_flat<float, kReduceUnroll, true>);
  (void)cudaGetLastError();
}

template <typename T>
bool vector_path_ok(const void* logits, int64_t row_stride, int V) {
  return ((reinterpret_cast<uintptr_t>(logits) & 15u) == 0) && ((row_stride * (int64_t)sizeof(T)) % 16 == 0) &&
         (V >= fly::Seg<T>::kElems * 32);
}

// Launches the row reduction.  `tail` carries the acceptance scan's arguments (tickets == NULL: no scan in
// this launch); its geometry fields are filled in here and returned through it for a stand-alone scan.
template <typename T>
cudaError_t launch_reduce(int sm_count, const void* logits, int64_t row_stride, int V, int64_t rows, int forced, int cap,
                          fly::Partial* partials, cudaStream_t st, fly::ScanParams* tail, float scale,
                          bool inputs_ready) {
  constexpr int kE = fly::Seg<T>::kElems;
  const bool vec = vector_path_ok<T>(logits, row_stride, V);
  const int64_t n = vec ? V / kE : V;
  const int64_t min_units = vec ? kMinBlockBytes / 16 : kMinBlockBytes / (int64_t)sizeof(T);
  const int64_t stride_units = (int64_t)fly::kReduceWarps * kReduceUnroll * 32;
  const FlatPlan pl = plan_flat(sm_count, rows, n, min_units, stride_units, cap, inputs_ready, forced);
  fly::ReducePlan g;
  g.n = n; g.span = pl.span; g.Q = pl.Q; g.total = rows * pl.span; g.slots = pl.slots;
  g.pieces = pl.Q < (1 << 30) ? pl.pieces : 0; g.V = V; g.row_stride = row_stride;
  g.scale = scale; g.wait_first = inputs_ready ? 0 : 1;
  tail->splits = pl.slots;
  tail->units_per_row = n;
  tail->row_span = pl.span;
  tail->Q = pl.Q;
  tail->scale = scale;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  fill_launch(&cfg, attr, (unsigned)pl.grid, fly::kReduceThreads, st, true);
  cfg.dynamicSmemBytes = vec ? kReduceRingBytes : 0;
  if (vec)
    return cudaLaunchKernelEx(&cfg, fly::reduce_rows_flat<T, kReduceUnroll, true>, static_cast<const T*>(logits), g, partials,
                              *tail);
  return cudaLaunchKernelEx(&cfg, fly::reduce_rows_flat<T, kReduceUnroll, false>, static_cast<const T*>(logits), g, partials,
                            *tail);
}

// The current device must be the one the pointers belong to (its ordinal is `device`).
cudaError_t launch_reduce_any(int device, fly_dtype_t dt, int sm_count, const void* logits, int64_t row_stride, int V,
                              int64_t rows, int forced, int cap, fly::Partial* partials, cudaStream_t st,
                              fly::ScanParams* tail, float scale, bool inputs_ready) {
  ensure_reduce_attrs(device);
  if (dt == FLY_BF16)
    return launch_reduce<__nv_bfloat16>(sm_count, logits, row_stride, V, rows, forced, cap, partials, st, tail, scale,
                                        inputs_ready);
  return launch_reduce<float>(sm_count, logits, row_stride, V, rows, forced, cap, partials, st, tail, scale, inputs_ready);
}

cudaError_t launch_scan(const fly::ScanParams& p, cudaStream_t st) {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  fill_launch(&cfg, attr, (unsigned)((p.B + fly::kScanWarps - 1) / fly::kScanWarps), fly::kScanThreads, st, true);
  return cudaLaunchKernelEx(&cfg, fly::scan_sequences, p);
}

fly_status_t check_args(const fly_verify* h, const fly_verify_args_t* a) {
  if (!h || !a) return FLY_ERR_INVALID_ARG;
  if (a->B < 1 || a->B > h->cfg.max_batch) return FLY_ERR_INVALID_ARG;
  if (a->K < 1 || a->K > h->cfg.max_k) return FLY_ERR_INVALID_ARG;
  if (!a->draft || !a->accept_len || !a->out_tokens) return FLY_ERR_INVALID_ARG;
  if (a->W < 0) return FLY_ERR_INVALID_ARG;
  if (std::isnan(a->theta)) return FLY_ERR_INVALID_ARG;
  if (a->theta_unit != FLY_THETA_NATS && a->theta_unit != FLY_THETA_NORMALIZED) return FLY_ERR_INVALID_ARG;
  if (!(a->temperature == 0.0 || (a->temperature >= 1e-6 && a->temperature <= 1e6))) return FLY_ERR_INVALID_ARG;
  if (a->inputs_ready != 0 && a->inputs_ready != 1) return FLY_ERR_INVALID_ARG;
  if (a->boundary != FLY_BOUNDARY_REJECT && a->boundary != FLY_BOUNDARY_CARRY) return FLY_ERR_INVALID_ARG;
  const bool has_logits = a->logits != nullptr;
  const bool has_fused = a->hidden != nullptr || a->weight != nullptr;
  if (has_logits == has_fused) return FLY_ERR_INVALID_ARG;
  if (has_fused && (!a->hidden || !a->weight)) return FLY_ERR_INVALID_ARG;
  if (has_logits && a->row_stride != 0 && a->row_stride < h->cfg.vocab) return FLY_ERR_INVALID_ARG;
  if (a->boundary == FLY_BOUNDARY_CARRY) {
    if (!a->state_out) return FLY_ERR_INVALID_ARG;
    if (a->W > a->K) return FLY_ERR_UNSUPPORTED;
  } else if (a->state_in) {
    return FLY_ERR_INVALID_ARG;  // the paper's rule has no cross-round state
  }
  return FLY_OK;
}

// log2(e) / T: turns a logit into the base-2 exponent of its softmax weight at temperature T (0 = 1).
float exponent_scale(double temperature) {
  const double T = temperature == 0.0 ? 1.0 : temperature;
  return (float)(1.4426950408889634 / T);
}

fly::ScanParams scan_params(const fly_verify* h, const fly_verify_args_t* a, const fly::Partial* partials, int splits);

// 2-D bf16 tensor map with the 128-byte swizzle: dims {inner, outer}, row pitch in bytes, box {64, box_rows}.
bool encode_map(fly_verify* h, CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint64_t pitch_bytes,
                uint32_t box_rows) {
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = h->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box,
                                     estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Fused LM-head step: one GEMM + row-statistics launch per block of up to 288
// positions, then the acceptance scan over the per-CTA partial states.
fly_status_t run_fused(fly_verify* h, const fly_verify_args_t* a, cudaStream_t st) {
  namespace L = fly::lmhead;
  const int V = h->cfg.vocab, D = h->cfg.hidden;
  const int64_t rows = (int64_t)a->B * (a->K + 1);
  if ((reinterpret_cast<uintptr_t>(a->hidden) & 15u) || (reinterpret_cast<uintptr_t>(a->weight) & 15u))
    return FLY_ERR_UNSUPPORTED;  // TMA needs 16-byte aligned bases
  if (h->map_w_ptr != a->weight) {
    const bool ok = h->weight_vd ? encode_map(h, &h->map_w, a->weight, (uint64_t)D, (uint64_t)V, (uint64_t)D * 2, L::kBlockV)
                                 : encode_map(h, &h->map_w, a->weight, (uint64_t)V, (uint64_t)D, (uint64_t)V * 2, 64);
    if (!ok) return FLY_ERR_CUDA;
    h->map_w_ptr = a->weight;
  }
  if (h->map_h_ptr != a->hidden || h->map_h_rows != rows) {
    if (!encode_map(h, &h->map_h, a->hidden, (uint64_t)D, (uint64_t)rows, (uint64_t)D * 2, L::kBoxPos)) return FLY_ERR_CUDA;
    h->map_h_ptr = a->hidden;
    h->map_h_rows = rows;
  }
  const int num_tiles = (V + L::kPairV - 1) / L::kPairV;  // one tile = 256 vocabulary entries = one CTA pair
  const int grid = 2 * (num_tiles < h->lm_pairs ? num_tiles : h->lm_pairs);
  for (int64_t row0 = 0; row0 < rows; row0 += L::kMaxPos) {
    L::Params p;
    p.R = (int)(rows - row0 < L::kMaxPos ? rows - row0 : L::kMaxPos);
    const int r16 = (p.R + 15) / 16 * 16;
    p.n0 = r16 < L::kHalfN ? r16 : L::kHalfN;
    p.n1 = r16 > L::kHalfN ? r16 - L::kHalfN : 0;
    p.V = V; p.D = D;
    p.num_tiles = num_tiles;
    p.num_kb = (D + L::kBlockK - 1) / L::kBlockK;
    p.row0 = (int)row0;
    p.w_kmajor = h->weight_vd;
    p.scale = exponent_scale(a->temperature);
    p.partials = h->lm_partials;
    p.status = h->lm_status;
    L::lmhead_verify_kernel<<<grid, L::kThreads, L::kSmemBytes, st>>>(h->map_w, h->map_h, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->last_launches++;
  }
  cudaError_t e;
  {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    const unsigned warps = fly::kFoldThreads / 32;
    fill_launch(&cfg, attr, (unsigned)((rows + warps - 1) / warps), fly::kFoldThreads, st, true);
    e = cudaLaunchKernelEx(&cfg, fly::fold_partials, (const fly::Partial*)h->lm_partials, grid, (int64_t)grid,
                           (int64_t)1, h->lm_folded, (int)rows, 0, exponent_scale(a->temperature), (int64_t)0, (int64_t)0);
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->last_launches++;
  }
  fly::ScanParams sp = scan_params(h, a, h->lm_folded, 1);
  sp.status = h->lm_status;  // a step whose GEMM kernel gave up is marked row by row, in stream order
  e = launch_scan(sp, st);
  if (e != cudaSuccess) return cuda_fail(h, e);
  h->last_launches++;
  return FLY_OK;
}

float theta_to_nats(const fly_verify* h, const fly_verify_args_t* a) {
  double th = a->theta;
  if (a->theta_unit == FLY_THETA_NORMALIZED) th *= std::log((double)h->cfg.vocab);
  return (float)th;
}

fly::ScanParams scan_params(const fly_verify* h, const fly_verify_args_t* a, const fly::Partial* partials, int splits) {
  fly::ScanParams p;
  p.B = a->B; p.K = a->K; p.V = h->cfg.vocab; p.splits = splits;
  p.units_per_row = 0; p.row_span = 0; p.Q = 0;  // every row has exactly `splits` parts unless the row reduction says otherwise
  p.scale = exponent_scale(a->temperature);
  p.partials = partials;
  p.tickets = nullptr;
  p.draft = a->draft;
  p.theta_nats = theta_to_nats(h, a);
  p.W = a->W > 64 ? 64 : a->W;
  p.carry = a->boundary == FLY_BOUNDARY_CARRY;
  p.state_in = reinterpret_cast<const int32_t*>(a->state_in);
  p.state_out = reinterpret_cast<int32_t*>(a->state_out);
  p.accept_len = a->accept_len;
  p.rollback = a->rollback;
  p.out_tokens = a->out_tokens;
  p.target_argmax = a->target_argmax;
  p.entropy = a->entropy;
  p.row_flags = a->row_flags;
  p.target_tokens = a->target_tokens;
  p.status = nullptr;
  return p;
}

}  // namespace

extern "C" {

const char* fly_status_string(fly_status_t s) {
  switch (s) {
    case FLY_OK: return "ok";
    case FLY_ERR_INVALID_ARG: return "invalid argument";
    case FLY_ERR_UNSUPPORTED: return "unsupported request";
    case FLY_ERR_CUDA: return "CUDA runtime error";
    case FLY_ERR_TIMEOUT: return "device-side wait timed out";
    case FLY_ERR_TOO_LARGE:
      return "step exceeds the built-in scratch area (B <= 1024, B*(K+1) <= 16384)";
  }
  return "unknown status";
}

fly_status_t fly_verify_create(const fly_verify_config_t* c, fly_verify_t** out) {
  if (out) *out = nullptr;
  if (!c || !out) return FLY_ERR_INVALID_ARG;
  if (c->max_batch < 1 || c->max_k < 1 || c->max_k > kMaxK || c->vocab < 1 || c->hidden < 0 || c->device < 0)
    return FLY_ERR_INVALID_ARG;
  if (c->logits_dtype != FLY_F32 && c->logits_dtype != FLY_BF16) return FLY_ERR_INVALID_ARG;
  // the fused path streams both operands with TMA: row pitches must be multiples of 16 bytes
  if (c->hidden > 0 && (c->hidden % 8 != 0 || c->vocab % 8 != 0)) return FLY_ERR_UNSUPPORTED;
  fly_verify* h = new (std::nothrow) fly_verify();
  if (!h) return FLY_ERR_INVALID_ARG;
  h->cfg = *c;
  h->max_rows = (int64_t)c->max_batch * (c->max_k + 1);
  DeviceGuard g(c->device);
  if (!g.ok) { delete h; return FLY_ERR_CUDA; }
  int sms = 0;
  cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
  if (e != cudaSuccess) { delete h; return FLY_ERR_CUDA; }
  h->sm_count = sms > 0 ? sms : 148;
  e = cudaMalloc(&h->partials, (size_t)h->max_rows * kMaxSplits * sizeof(fly::Partial));
  if (e != cudaSuccess) { delete h; return FLY_ERR_CUDA; }
  e = cudaMalloc(&h->tickets, (size_t)c->max_batch * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(h->tickets, 0, (size_t)c->max_batch * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMalloc(&h->lm_status, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(h->lm_status, 0, sizeof(int));
  if (e == cudaSuccess) e = cudaMalloc(&h->lm_folded, (size_t)h->max_rows * sizeof(fly::Partial));
  if (e != cudaSuccess) {
    cudaFree(h->partials); cudaFree(h->tickets); cudaFree(h->lm_status); cudaFree(h->lm_folded);
    delete h;
    return FLY_ERR_CUDA;
  }
  if (c->hidden > 0) {
    e = cudaMalloc(&h->lm_partials, (size_t)h->max_rows * h->sm_count * sizeof(fly::Partial));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(fly::lmhead::lmhead_verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               fly::lmhead::kSmemBytes);
    if (e == cudaSuccess) {
      // how many pairs (clusters of two CTAs, one CTA per SM) fit on the device at once
      cudaLaunchConfig_t lc;
      memset(&lc, 0, sizeof(lc));
      lc.gridDim = dim3((unsigned)(h->sm_count & ~1));
      lc.blockDim = dim3(fly::lmhead::kThreads);
      lc.dynamicSmemBytes = fly::lmhead::kSmemBytes;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.attrs = at;
      lc.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, fly::lmhead::lmhead_verify_kernel, &lc) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        n = h->sm_count / 2;
      }
      h->lm_pairs = n < h->sm_count / 2 ? n : h->sm_count / 2;
      if (h->lm_pairs < 1) h->lm_pairs = 1;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (e == cudaSuccess) e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || !fn) {
      fly_status_t st = cuda_fail(h, e);
      (void)st;
      cudaFree(h->partials); cudaFree(h->tickets); cudaFree(h->lm_partials); cudaFree(h->lm_folded);
      cudaFree(h->lm_status);
      delete h;
      return FLY_ERR_CUDA;
    }
    h->encode_tiled = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
  }
  *out = h;
  return FLY_OK;
}

fly_status_t fly_verify_destroy(fly_verify_t* h) {
  if (!h) return FLY_OK;
  DeviceGuard g(h->cfg.device);
  if (g.ok) {
    cudaFree(h->partials);
    cudaFree(h->tickets);
    cudaFree(h->lm_partials);
    cudaFree(h->lm_folded);
    cudaFree(h->lm_status);
    cudaFree(h->st_hidden);
    cudaFree(h->st_logits);
    cudaFree(h->st_ints);
    cudaFreeHost(h->st_host);
  }
  delete h;
  return FLY_OK;
}

fly_status_t fly_verify_set_option(fly_verify_t* h, fly_option_t opt, int32_t v) {
  if (!h) return FLY_ERR_INVALID_ARG;
  switch (opt) {
    case FLY_OPT_SPLITS:
      if (v < 0 || v > kMaxSplits) return FLY_ERR_INVALID_ARG;
      h->forced_splits = v;
      return FLY_OK;
    case FLY_OPT_SCAN_MODE:
      if (v != 0 && v != 1) return FLY_ERR_INVALID_ARG;
      h->scan_mode = v;
      return FLY_OK;
    case FLY_OPT_WEIGHT_LAYOUT:
      if (v != 0 && v != 1) return FLY_ERR_INVALID_ARG;
      h->weight_vd = v;
      h->map_w_ptr = nullptr;  // the cached tensor map describes the other layout
      return FLY_OK;
  }
  return FLY_ERR_INVALID_ARG;
}

fly_status_t fly_verify_reduce_shard(fly_verify_t* h, int32_t rows, const void* logits, int64_t row_stride,
                                     int32_t vocab_offset, double temperature, fly_partial_t* partial_out,
                                     void* cuda_stream) {
  if (!h || !logits || !partial_out) return FLY_ERR_INVALID_ARG;
  if (rows < 1 || rows > h->max_rows || vocab_offset < 0) return FLY_ERR_INVALID_ARG;
  if (!(temperature == 0.0 || (temperature >= 1e-6 && temperature <= 1e6))) return FLY_ERR_INVALID_ARG;
  const int V = h->cfg.vocab;
  if (row_stride != 0 && row_stride < V) return FLY_ERR_INVALID_ARG;
  if ((int64_t)vocab_offset + V > 0x7fffffff) return FLY_ERR_INVALID_ARG;
  DeviceGuard g(h->cfg.device);
  if (!g.ok) return FLY_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t stride = row_stride ? row_stride : V;
  const float scale = exponent_scale(temperature);
  fly::ScanParams none;
  memset(&none, 0, sizeof(none));  // tickets == NULL: no acceptance scan in this launch
  cudaError_t e = launch_reduce_any(h->cfg.device, h->cfg.logits_dtype, h->sm_count, logits, stride, V, rows, h->forced_splits, kMaxSplits,
                                    h->partials, st, &none, scale, false);
  if (e != cudaSuccess) return cuda_fail(h, e);
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  const unsigned warps = fly::kFoldThreads / 32;
  fill_launch(&cfg, attr, (unsigned)((rows + warps - 1) / warps), fly::kFoldThreads, st, true);
  e = cudaLaunchKernelEx(&cfg, fly::fold_partials, (const fly::Partial*)h->partials, none.splits, (int64_t)none.splits,
                         (int64_t)1, reinterpret_cast<fly::Partial*>(partial_out), (int)rows, (int)vocab_offset, scale,
                         none.row_span, none.Q);
  if (e != cudaSuccess) return cuda_fail(h, e);
  h->last_launches = 2;
  return FLY_OK;
}

fly_status_t fly_verify_run_partials(fly_verify_t* h, const fly_verify_args_t* a, const fly_partial_t* partials,
                                     int32_t world, int32_t total_vocab, void* cuda_stream) {
  if (!h || !a || !partials || world < 1 || world > 1024 || total_vocab < 1) return FLY_ERR_INVALID_ARG;
  if (a->logits || a->hidden || a->weight) return FLY_ERR_INVALID_ARG;  // the logits were reduced by the shards
  fly_verify_args_t chk = *a;
  chk.logits = partials;  // satisfies the "exactly one input" rule of the common checks
  fly_status_t s = check_args(h, &chk);
  if (s != FLY_OK) return s;
  DeviceGuard g(h->cfg.device);
  if (!g.ok) return FLY_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t rows = (int64_t)a->B * (a->K + 1);
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  const unsigned warps = fly::kFoldThreads / 32;
  fill_launch(&cfg, attr, (unsigned)((rows + warps - 1) / warps), fly::kFoldThreads, st, false);
  // all-gather layout: [world, rows]
  cudaError_t e = cudaLaunchKernelEx(&cfg, fly::fold_partials, reinterpret_cast<const fly::Partial*>(partials), (int)world,
                                     (int64_t)1, (int64_t)rows, h->lm_folded, (int)rows, 0, exponent_scale(a->temperature),
                                     (int64_t)0, (int64_t)0);
  if (e != cudaSuccess) return cuda_fail(h, e);
  fly::ScanParams sp = scan_params(h, a, h->lm_folded, 1);
  sp.V = total_vocab;
  double th = a->theta;
  if (a->theta_unit == FLY_THETA_NORMALIZED) th *= std::log((double)total_vocab);
  sp.theta_nats = (float)th;
  e = launch_scan(sp, st);
  if (e != cudaSuccess) return cuda_fail(h, e);
  h->last_launches = 2;
  return FLY_OK;
}

fly_status_t fly_pld_draft(int32_t device, int32_t B, const int32_t* tokens, int64_t stride, const int32_t* lengths,
                           int32_t max_ngram, int32_t min_ngram, int32_t K, int32_t* draft, int32_t* count,
                           int32_t* match_pos, int32_t* match_ngram, void* cuda_stream) {
  if (device < 0 || B < 1 || !tokens || !lengths || !draft || !count || stride < 1) return FLY_ERR_INVALID_ARG;
  if (min_ngram < 1 || max_ngram < min_ngram || max_ngram > fly::pld::kMaxNgram || K < 1) return FLY_ERR_INVALID_ARG;
  DeviceGuard g(device);
  if (!g.ok) return FLY_ERR_CUDA;
  fly::pld::Params p;
  p.tokens = tokens; p.stride = stride; p.lengths = lengths;
  p.B = B; p.max_ngram = max_ngram; p.min_ngram = min_ngram; p.K = K;
  p.draft = draft; p.count = count; p.match_pos = match_pos; p.match_ngram = match_ngram;
  fly::pld::pld_draft_kernel<<<(unsigned)B, fly::pld::kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? FLY_OK : FLY_ERR_CUDA;
}

fly_status_t fly_verify_device_status(fly_verify_t* h, void* cuda_stream) {
  if (!h) return FLY_ERR_INVALID_ARG;
  DeviceGuard g(h->cfg.device);
  if (!g.ok) return FLY_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  int word = 0;
  if (h->lm_status) {
    if ((e = cudaMemcpyAsync(&word, h->lm_status, sizeof(int), cudaMemcpyDeviceToHost, st)) != cudaSuccess)
      return cuda_fail(h, e);
  }
  if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(h, e);
  if (word != 0) {
    if ((e = cudaMemsetAsync(h->lm_status, 0, sizeof(int), st)) != cudaSuccess) return cuda_fail(h, e);
    return FLY_ERR_TIMEOUT;
  }
  return FLY_OK;
}

fly_status_t fly_verify_selftest_wait(fly_verify_t* h, void* cuda_stream) {
  if (!h) return FLY_ERR_INVALID_ARG;
  DeviceGuard g(h->cfg.device);
  if (!g.ok) return FLY_ERR_CUDA;
  fly::lmhead::wait_selftest_kernel<<<1, 1, 0, static_cast<cudaStream_t>(cuda_stream)>>>(h->lm_status, 2000000ull);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? FLY_OK : cuda_fail(h, e);
}

fly_status_t fly_verify_plan(int32_t sm_count, int64_t rows, int32_t vocab, fly_dtype_t dtype, int32_t vector_path,
                             int32_t inputs_ready, int32_t forced_pieces, fly_plan_t* out) {
  if (!out || sm_count < 1 || rows < 1 || rows > (int64_t)1 << 24 || vocab < 1) return FLY_ERR_INVALID_ARG;
  if (dtype != FLY_F32 && dtype != FLY_BF16) return FLY_ERR_INVALID_ARG;
  if (forced_pieces < 0 || forced_pieces > kMaxSplits) return FLY_ERR_INVALID_ARG;
  const int64_t esz = dtype == FLY_BF16 ? 2 : 4;
  const int64_t per_seg = 16 / esz;
  if (vector_path && vocab < per_seg * 32) return FLY_ERR_INVALID_ARG;
  const int64_t n = vector_path ? vocab / per_seg : vocab;
  const int64_t min_units = vector_path ? kMinBlockBytes / 16 : kMinBlockBytes / esz;
  const FlatPlan pl = plan_flat(sm_count, rows, n, min_units, (int64_t)fly::kReduceWarps * kReduceUnroll * 32, kMaxSplits,
                                inputs_ready != 0, forced_pieces);
  out->grid = pl.grid;
  out->slots = pl.slots;
  out->units_per_block = pl.Q;
  out->units_per_row = n;
  out->row_span = pl.span;
  return FLY_OK;
}

int32_t fly_verify_last_launch_count(const fly_verify_t* h) { return h ? h->last_launches : 0; }
int32_t fly_verify_last_cuda_error(const fly_verify_t* h) { return h ? h->last_cuda_error : 0; }

fly_status_t fly_verify_run(fly_verify_t* h, const fly_verify_args_t* a, void* cuda_stream) {
  fly_status_t s = check_args(h, a);
  if (s != FLY_OK) return s;
  if (!a->logits && h->cfg.hidden <= 0) return FLY_ERR_INVALID_ARG;  // the handle was created without a hidden size
  DeviceGuard g(h->cfg.device);
  if (!g.ok) return FLY_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int V = h->cfg.vocab;
  const int64_t rows = (int64_t)a->B * (a->K + 1);
  const int64_t stride = a->row_stride ? a->row_stride : V;
  h->last_launches = 0;
  if (!a->logits) return run_fused(h, a, st);

  fly::ScanParams p = scan_params(h, a, h->partials, 1);
  // The acceptance scan runs as the tail of the reduction (the block that completes a sequence verifies it) unless
  // the handle asks for a kernel of its own.  Measured in plain stream order the two cost the same; the tail also
  // lets consecutive steps overlap (inputs_ready) and keeps a step at one launch.
  const bool fused_tail = h->scan_mode == 0;
  p.tickets = fused_tail ? h->tickets : nullptr;
  cudaError_t e = launch_reduce_any(h->cfg.device, h->cfg.logits_dtype, h->sm_count, a->logits, stride, V, rows, h->forced_splits,
                                    kMaxSplits, h->partials, st, &p, p.scale, a->inputs_ready != 0);
  if (e != cudaSuccess) return cuda_fail(h, e);
  h->last_launches++;
  if (!fused_tail) {
    e = launch_scan(p, st);
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->last_launches++;
  }
  return FLY_OK;
}

fly_status_t fly_verify_run_host(fly_verify_t* h, const fly_verify_args_t* a, void* cuda_stream) {
  fly_status_t s = check_args(h, a);
  if (s != FLY_OK) return s;
  if (!a->logits && h->cfg.hidden <= 0) return FLY_ERR_INVALID_ARG;
  DeviceGuard g(h->cfg.device);
  if (!g.ok) return FLY_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int V = h->cfg.vocab;
  const size_t esz = h->cfg.logits_dtype == FLY_BF16 ? 2 : 4;
  const int64_t K1 = a->K + 1, B = a->B, rows = B * K1;
  const int64_t stride = a->row_stride ? a->row_stride : V;
  cudaError_t e;
  if (!h->st_ints) {
    // staging sized once for the largest run this handle allows: the small inputs and all outputs are
    // packed into one block each way, so that a step costs one small copy in and one out
    const int64_t mb = h->cfg.max_batch, mk1 = h->cfg.max_k + 1;
    const size_t words = (size_t)(mb * (mk1 - 1) + 3 * mb + mb * mk1) + (size_t)(3 * mb + mb + mb + 4 * mb * mk1);
    int32_t* dev_block = nullptr;
    int32_t* host_block = nullptr;
    if ((e = cudaMalloc(&dev_block, words * sizeof(int32_t))) != cudaSuccess) {
      (void)cudaGetLastError();
      return cuda_fail(h, e);
    }
    if ((e = cudaMallocHost(&host_block, words * sizeof(int32_t))) != cudaSuccess) {
      (void)cudaGetLastError();
      cudaFree(dev_block);
      return cuda_fail(h, e);
    }
    h->st_ints = dev_block;  // both or neither
    h->st_host = host_block;
  }
  const size_t hidden_bytes = a->logits ? 0 : (size_t)rows * h->cfg.hidden * 2;
  if (hidden_bytes > h->st_hidden_bytes) {
    cudaFree(h->st_hidden);
    h->st_hidden = nullptr;
    h->st_hidden_bytes = 0;
    if ((e = cudaMalloc(&h->st_hidden, hidden_bytes)) != cudaSuccess) return cuda_fail(h, e);
    h->st_hidden_bytes = hidden_bytes;
  }
  const size_t logit_bytes = a->logits ? (size_t)(((rows - 1) * stride + V)) * esz : 0;
  if (logit_bytes > h->st_logits_bytes) {
    cudaFree(h->st_logits);
    h->st_logits = nullptr;
    h->st_logits_bytes = 0;
    if ((e = cudaMalloc(&h->st_logits, logit_bytes)) != cudaSuccess) return cuda_fail(h, e);
    h->st_logits_bytes = logit_bytes;
  }
  // word offsets inside the staging block (same layout on the host and on the device)
  const int64_t o_draft = 0, o_state_in = o_draft + B * a->K, o_target = o_state_in + 3 * B, in_words = o_target + rows;
  const int64_t o_state_out = in_words, o_accept = o_state_out + 3 * B, o_rollback = o_accept + B,
                o_tokens = o_rollback + B, o_argmax = o_tokens + rows, o_flags = o_argmax + rows,
                o_entropy = o_flags + rows, all_words = o_entropy + rows;
  int32_t* dv = h->st_ints;
  int32_t* hv = h->st_host;
  memcpy(hv + o_draft, a->draft, (size_t)(B * a->K) * 4);
  if (a->state_in) memcpy(hv + o_state_in, a->state_in, (size_t)B * 12);
  if (a->target_tokens) memcpy(hv + o_target, a->target_tokens, (size_t)rows * 4);

  if (a->logits && (e = cudaMemcpyAsync(h->st_logits, a->logits, logit_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return cuda_fail(h, e);
  if (!a->logits && (e = cudaMemcpyAsync(h->st_hidden, a->hidden, hidden_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess)
    return cuda_fail(h, e);
  if ((e = cudaMemcpyAsync(dv, hv, (size_t)in_words * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(h, e);

  fly_verify_args_t d = *a;
  d.logits = a->logits ? h->st_logits : nullptr;
  d.hidden = a->logits ? nullptr : h->st_hidden;  // the weight stays where it is: device memory
  d.draft = dv + o_draft;
  d.state_in = a->state_in ? reinterpret_cast<const fly_state_t*>(dv + o_state_in) : nullptr;
  d.state_out = reinterpret_cast<fly_state_t*>(dv + o_state_out);
  d.accept_len = dv + o_accept;
  d.rollback = dv + o_rollback;
  d.out_tokens = dv + o_tokens;
  d.target_argmax = dv + o_argmax;
  d.entropy = reinterpret_cast<float*>(dv + o_entropy);
  d.row_flags = reinterpret_cast<uint32_t*>(dv + o_flags);
  d.target_tokens = a->target_tokens ? dv + o_target : nullptr;
  s = fly_verify_run(h, &d, cuda_stream);
  if (s != FLY_OK) return s;

  if ((e = cudaMemcpyAsync(hv + in_words, dv + in_words, (size_t)(all_words - in_words) * 4, cudaMemcpyDeviceToHost, st)) !=
      cudaSuccess)
    return cuda_fail(h, e);
  if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(h, e);
  auto back = [&](void* dst, int64_t off, size_t bytes) {
    if (dst) memcpy(dst, hv + off, bytes);
  };
  back(a->accept_len, o_accept, (size_t)B * 4);
  back(a->rollback, o_rollback, (size_t)B * 4);
  back(a->out_tokens, o_tokens, (size_t)rows * 4);
  back(a->target_argmax, o_argmax, (size_t)rows * 4);
  back(a->entropy, o_entropy, (size_t)rows * 4);
  back(a->row_flags, o_flags, (size_t)rows * 4);
  back(a->state_out, o_state_out, (size_t)B * 12);
  return FLY_OK;
}

// ---------------------------------------------------------------------------
// fly_verify_run_static: the logits-path step for callers that cannot allocate.
// Its scratch is this array in the library image.  In host code the array's
// name is only a handle for the runtime, not a device address: the address is
// looked up once per device with cudaGetSymbolAddress and handed to the kernel
// like any other scratch pointer.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_fly_static_scratch[FLY_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kStaticMaxDevices = 64;
struct StaticSlot {
  void* base = nullptr;  // device address of g_fly_static_scratch on this device
  int sm_count = 0;
};
StaticSlot g_static_slots[kStaticMaxDevices];
std::mutex g_static_mu;

// Once per device, with that device current.
cudaError_t static_scratch_for(int device, StaticSlot* out) {
  std::lock_guard<std::mutex> lock(g_static_mu);
  StaticSlot& s = g_static_slots[device];
  if (!s.base) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_fly_static_scratch);
    if (e != cudaSuccess) return e;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return e;
    s.sm_count = sms > 0 ? sms : 148;
    s.base = p;
  }
  *out = s;
  return cudaSuccess;
}

}  // namespace

fly_status_t fly_verify_run_static(int32_t device, int32_t vocab, fly_dtype_t logits_dtype,
                                   const fly_verify_args_t* a, void* cuda_stream) {
  if (!a || device < 0 || device >= kStaticMaxDevices || vocab < 1) return FLY_ERR_INVALID_ARG;
  if (logits_dtype != FLY_F32 && logits_dtype != FLY_BF16) return FLY_ERR_INVALID_ARG;
  if (a->B > FLY_STATIC_MAX_BATCH && a->K >= 1 && a->K <= kMaxK) return FLY_ERR_TOO_LARGE;
  fly_verify h;  // a stack stand-in for a handle: describes the step, owns nothing
  h.cfg.device = device;
  h.cfg.max_batch = FLY_STATIC_MAX_BATCH;
  h.cfg.max_k = kMaxK;
  h.cfg.vocab = vocab;
  h.cfg.logits_dtype = logits_dtype;
  h.cfg.hidden = 0;
  fly_status_t s = check_args(&h, a);
  if (s != FLY_OK) return s;
  if (!a->logits) return FLY_ERR_UNSUPPORTED;  // the fused LM-head path needs a handle
  const int64_t rows = (int64_t)a->B * (a->K + 1);
  if (rows > FLY_STATIC_MAX_PIECES) return FLY_ERR_TOO_LARGE;

  DeviceGuard g(device);
  if (!g.ok) return FLY_ERR_CUDA;
  StaticSlot slot;
  if (static_scratch_for(device, &slot) != cudaSuccess) return FLY_ERR_CUDA;
  unsigned int* tickets = static_cast<unsigned int*>(slot.base);
  fly::Partial* partials =
      reinterpret_cast<fly::Partial*>(static_cast<unsigned char*>(slot.base) + FLY_STATIC_MAX_BATCH * 4);
  h.sm_count = slot.sm_count;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t stride = a->row_stride ? a->row_stride : vocab;
  const int64_t room = FLY_STATIC_MAX_PIECES / rows;  // Partial slots per row that fit, >= 1
  const int cap = (int)(room < kMaxSplits ? room : kMaxSplits);

  fly::ScanParams p = scan_params(&h, a, partials, 1);
  p.tickets = tickets;

  // The arrival counters must start at zero, whatever an earlier call left behind.
  cudaError_t e = cudaMemsetAsync(tickets, 0, (size_t)a->B * 4, st);
  if (e != cudaSuccess) return FLY_ERR_CUDA;
  e = launch_reduce_any(device, logits_dtype, h.sm_count, a->logits, stride, vocab, rows, 0, cap, partials, st, &p, p.scale,
                        a->inputs_ready != 0);
  return e == cudaSuccess ? FLY_OK : FLY_ERR_CUDA;
}

}  // extern "C"

// Acceptance scan of the FLy verification step: one warp per sequence.  It runs
// either as the tail of the row-reduction kernel (the last block to finish a
// sequence's rows does it) or as a launch of its own.
//
// Lanes first fold the per-unit Partials of "their" rows into entropy and
// greedy token, then the warp forms the match bits Delta_i (Eq. 2) and the gate
// bits [H_i >= theta] (Eq. 6) with ballots and walks the mismatch set J in
// ascending order exactly as Algorithm 1 does (steps 3 and 4): Strict rejects,
// Defer looks at the next W positions (Eq. 8, Eq. 9), a window that does not
// fit in the round rejects (paper) or is carried to the next round (extension).
// Finally the lanes write the tokens to append (Algorithm 1's concat lines).
#pragma once
#include "fly_common.cuh"

namespace fly {

constexpr int kScanThreads = 128;
constexpr int kScanWarps = kScanThreads / 32;
constexpr int kMaxRows = 64;  // K + 1 <= 64

struct ScanParams {
  int B, K, V;
  int splits;               // Partial slots per row
  // Flat partition of the row reduction (Q > 0): a row holds units_per_row units and spans row_span >= units_per_row
  // positions of the flat index space; thread block b reduced the flat range [b*Q, (b+1)*Q), so row r has
  // ((r+1)*span - 1)/Q - (r*span)/Q + 1 pieces in its first slots.  Q == 0: every row has exactly `splits` pieces.
  int64_t units_per_row;
  int64_t row_span;
  int64_t Q;
  float scale;              // log2(e) / temperature (exponent unit of the partial states)
  const Partial* partials;  // [B*(K+1), splits]
  unsigned int* tickets;    // [B] arrival counters for the fused tail (zero between launches), or null
  const int32_t* draft;     // [B, K]
  float theta_nats;
  int W;
  int carry;                // 0: paper rule at the round boundary, 1: carry extension
  const int32_t* state_in;  // [B, 3] or null
  int32_t* state_out;       // [B, 3] or null
  int32_t* accept_len;      // [B]
  int32_t* rollback;        // [B] or null
  int32_t* out_tokens;      // [B, K+1]
  int32_t* target_argmax;   // [B, K+1] or null
  float* entropy;           // [B, K+1] or null
  uint32_t* row_flags;      // [B, K+1] or null
  const int32_t* target_tokens;  // [B, K+1] or null: the caller's y_i instead of the argmax
  const int* status;             // fused path: device word that is non-zero when a bounded wait of the GEMM kernel ran out
};

struct RoundOutcome {
  int s;         // accepted-token count, 1..K+1
  int rollback;  // tokens to remove first (revoked carry), else 0
  int revoke;    // 1: out_tokens = [correction]
  int st_pending, st_len, st_corr_pos;  // state_out; st_corr_pos = position j whose y_j is the correction (0: none)
};

// mism / defer: bit (i-1) set <=> position i is a mismatch / has H_i >= theta.
__device__ __forceinline__ RoundOutcome decide_round(uint64_t mism, uint64_t defer, int K, int W, int carry,
                                                     int pend_in, int len_in) {
  RoundOutcome o;
  o.s = K + 1; o.rollback = 0; o.revoke = 0; o.st_pending = 0; o.st_len = 0; o.st_corr_pos = 0;
  if (carry && pend_in > 0) {
    const uint64_t first_r = pend_in >= 64 ? ~0ull : ((1ull << pend_in) - 1ull);
    if (mism & first_r) {  // a mismatch inside the carried window: revoke
      o.s = 1; o.rollback = len_in; o.revoke = 1;
      return o;
    }
  }
  uint64_t rest = mism;
  while (rest) {
    const int j = __ffsll((long long)rest);  // 1-based position of the next mismatch
    rest &= rest - 1;
    if (!((defer >> (j - 1)) & 1ull)) { o.s = j; return o; }  // Strict
    // positions j+1 .. min(j+W, K)  <->  bits j .. min(j+W,K)-1
    const int hi = min(j + W, K);
    const uint64_t upto_hi = hi >= 64 ? ~0ull : ((1ull << hi) - 1ull);
    const uint64_t upto_j = (1ull << j) - 1ull;  // j <= K <= 63
    const uint64_t later = mism & upto_hi & ~upto_j;
    if (later == 0 && j + W <= K) continue;  // benign: keep the draft token
    if (later == 0 && carry) {               // window leaves the round clean: carry it
      o.s = K + 1; o.st_pending = j + W - K; o.st_len = K - j + 2; o.st_corr_pos = j;
      return o;
    }
    o.s = j;
    return o;
  }
  return o;
}

__device__ __forceinline__ Partial ld_partial_cg(const Partial* p) {
  // partial states are written by other thread blocks: read them through L2
  const int4 v = __ldcg(reinterpret_cast<const int4*>(p));
  Partial q;
  q.mx = __int_as_float(v.x); q.S = __int_as_float(v.y); q.u = __int_as_float(v.z); q.idx = v.w;
  return q;
}

// Number of pieces the flat partition cut row `row` into (see ScanParams).
__device__ __forceinline__ int pieces_of_row(int64_t row, int64_t span, int64_t Q, int fixed) {
  if (Q <= 0) return fixed;
  const int64_t f0 = row * span;
  return (int)((f0 + span - 1) / Q - f0 / Q) + 1;
}

// One warp verifies sequence b.  sm_y: kMaxRows ints of shared memory private to the warp.
__device__ __forceinline__ void scan_one_sequence(const ScanParams& p, int b, int lane, int* sm_y) {
  const int K = p.K, K1 = p.K + 1;
  uint64_t mism = 0, defer = 0;
  // Issue the loads that do not depend on the partial states first (draft tokens, carried state):
  // they are cold misses, and this is the tail of the step, where every dependent round trip counts.
  int dr[2];
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int i = half * 32 + lane;
    dr[half] = i < K ? p.draft[(int64_t)b * K + i] : 0;
  }
  int pend = 0, len = 0, corr = -1;
  // A fused step whose GEMM kernel gave up has no usable statistics: every row is flagged, nothing is accepted.
  const bool failed = p.status != nullptr && *reinterpret_cast<const volatile int*>(p.status) != 0;
  bool bad_state = false;
  if (p.carry && p.state_in) {
    pend = p.state_in[b * 3 + 0];
    len = p.state_in[b * 3 + 1];
    corr = p.state_in[b * 3 + 2];
    // The state is device data: only states this library writes are honoured (pending <= W <= K).  Anything
    // else is flagged and ignored, so that no token id out of range and no negative count can leave here.
    bad_state = pend < 0 || pend > K || len < 0 || (pend > 0 && (corr < 0 || corr >= p.V));
    if (bad_state) { pend = 0; len = 0; corr = -1; }
  }
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int i = half * 32 + lane;  // 0-based row of this sequence
    bool is_mism = false, is_defer = false;
    if (i < K1) {
      const int64_t row = (int64_t)b * K1 + i;
      const Partial* pp = p.partials + row * p.splits;
      const int pieces = pieces_of_row(row, p.row_span, p.Q, p.splits);
      Partial acc = empty_partial();
      for (int s0 = 0; s0 < pieces; s0 += 4) {  // four independent loads in flight
        Partial q[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) q[t] = (s0 + t < pieces) ? ld_partial_cg(pp + s0 + t) : empty_partial();
#pragma unroll
        for (int t = 0; t < 4; ++t) merge_partial(acc, q[t], p.scale);
      }
      // entropy is non-negative; rounding may leave -1e-7 on a one-hot row
      // lg2.approx and the fast division are good to ~1e-6 here (S >= 1 once a row has a finite entry); this is the
      // end of the step's critical path
      const float H = fmaxf(kLn2 * (lg2_approx(acc.S) - __fdividef(acc.u, acc.S)), 0.f);
      uint32_t flag = 0;
      if (!(fabsf(acc.S) <= 3.0e38f) || !(acc.mx <= 3.0e38f) || acc.mx <= kMaskFloor) flag |= kFlagNonFinite;
      if (failed) flag |= kFlagStepFailed;
      int y = acc.idx;
      if (flag || y < 0 || y >= p.V) y = 0;  // keep every emitted id in range
      const int greedy = y;
      if (p.target_tokens && !(flag & kFlagNonFinite)) {  // the caller drew y_i itself
        y = p.target_tokens[row];
        if (y < 0 || y >= p.V) { flag |= kFlagBadTarget; y = 0; }
      }
      sm_y[i] = y;
      if (i < K) {
        const int d = dr[half];
        if (d < 0 || d >= p.V) flag |= kFlagBadDraft;
        is_mism = (d != y) || flag;
        is_defer = (H >= p.theta_nats) && !flag;  // a flagged position is never kept
      }
      if (p.target_argmax) p.target_argmax[row] = greedy;
      if (p.entropy) p.entropy[row] = H;
      if (p.row_flags) p.row_flags[row] = flag | ((i == 0 && bad_state) ? kFlagBadState : 0u);
    }
    const uint64_t mb = __ballot_sync(0xffffffffu, is_mism);
    const uint64_t db = __ballot_sync(0xffffffffu, is_defer);
    mism |= mb << (32 * half);
    defer |= db << (32 * half);
  }
  __syncwarp();

  __syncwarp();  // state_in may alias state_out: all lanes have read it (above) before lane 0 writes
  const RoundOutcome o = decide_round(mism, defer, K, p.W, p.carry, pend, len);

#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int i = half * 32 + lane;
    if (i < K1) {
      int tok = -1;
      if (o.revoke) tok = (i == 0) ? corr : -1;
      else if (i < o.s - 1) tok = dr[half];
      else if (i == o.s - 1) tok = sm_y[i];
      p.out_tokens[(int64_t)b * K1 + i] = tok;
    }
  }
  if (lane == 0) {
    p.accept_len[b] = o.s;
    if (p.rollback) p.rollback[b] = o.rollback;
    if (p.state_out) {
      p.state_out[b * 3 + 0] = o.st_pending;
      p.state_out[b * 3 + 1] = o.st_len;
      p.state_out[b * 3 + 2] = o.st_corr_pos ? sm_y[o.st_corr_pos - 1] : -1;
    }
  }
}

// Folds the n partial states of every row into one (out[row]); one warp per row.  Part j of row r
// is in[r * row_stride + j * part_stride].  The fused LM-head kernel leaves one partial state per row
// and CTA, a vocabulary-parallel target one per row and rank; folding them with 32 lanes in parallel
// keeps the acceptance scan's per-lane loop short.  idx_offset is added to the winning index (a
// vocabulary shard reports global token ids).  With Q > 0 the number of parts of a row follows from
// the flat partition of the row reduction (see ScanParams) instead of being n_fixed.
constexpr int kFoldThreads = 128;
__global__ void __launch_bounds__(kFoldThreads) fold_partials(const Partial* __restrict__ in, int n_fixed, int64_t row_stride,
                                                              int64_t part_stride, Partial* __restrict__ out, int rows,
                                                              int idx_offset, float scale, int64_t row_span, int64_t Q) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (kFoldThreads / 32) + (threadIdx.x >> 5);
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the producer grid has completed
  asm volatile("griddepcontrol.launch_dependents;");
  if (row >= rows) return;
  const int n = pieces_of_row(row, row_span, Q, n_fixed);
  const Partial* src = in + (int64_t)row * row_stride;
  Partial acc = empty_partial();
  for (int j0 = 0; j0 < n; j0 += 128) {  // four independent loads in flight per lane
    Partial q[4];
#pragma unroll
    for (int t = 0; t < 4; ++t)
      q[t] = (j0 + t * 32 + lane < n) ? ld_partial_cg(src + (int64_t)(j0 + t * 32 + lane) * part_stride) : empty_partial();
#pragma unroll
    for (int t = 0; t < 4; ++t) merge_partial(acc, q[t], scale);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const Partial q = shfl_xor_partial(acc, o);
    merge_partial(acc, q, scale);
  }
  if (lane == 0) {
    if (acc.idx != kIdxNone) acc.idx += idx_offset;
    out[row] = acc;
  }
}

// Stand-alone launch: one warp per sequence, after the row reduction.
__global__ void __launch_bounds__(kScanThreads) scan_sequences(ScanParams p) {
  __shared__ int sm_y[kScanWarps][kMaxRows];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x * kScanWarps + warp;
  // every thread waits for the producer grid (row reduction) to complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (b >= p.B) return;
  scan_one_sequence(p, b, lane, sm_y[warp]);
}

}  // namespace fly

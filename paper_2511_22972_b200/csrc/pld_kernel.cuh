// Prompt-lookup drafting: the parameter-free n-gram retrieval with which the paper speeds up its
// drafter (Section 2.3, multi-level acceleration).  For one sequence of L tokens: take its last n
// tokens as the query, find the EARLIEST earlier position p < L - n where the same n tokens occur,
// and propose the tokens that followed them, tokens[p+n .. p+n+K) cut at L.  n runs from max_ngram
// down to min_ngram; the first n with a match wins.  No match: count = 0.
//
// One thread block per sequence.  Threads test candidate positions in parallel (the query's n <= 8
// tokens live in registers), a block-wide minimum picks the earliest match, and the K continuation
// tokens are copied out.  The work is a single pass over L int32 per tried n: a few KB per sequence.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fly {
namespace pld {

constexpr int kThreads = 256;
constexpr int kMaxNgram = 8;

struct Params {
  const int32_t* tokens;   // [B, stride]
  int64_t stride;
  const int32_t* lengths;  // [B]
  int B, max_ngram, min_ngram, K;
  int32_t* draft;          // [B, K], -1 where nothing is proposed
  int32_t* count;          // [B]
  int32_t* match_pos;      // [B] or null: p, -1 if no match
  int32_t* match_ngram;    // [B] or null: n, 0 if no match
};

__global__ void __launch_bounds__(kThreads) pld_draft_kernel(const Params p) {
  __shared__ int best[kThreads / 32];
  __shared__ int found_pos;
  const int b = blockIdx.x;
  const int32_t* tok = p.tokens + (int64_t)b * p.stride;
  // lengths is device data: a value outside [0, stride] must not steer any load past the sequence's row.
  // Such a sequence proposes nothing (count 0, match_pos -1), as an empty one does.
  const int Lraw = p.lengths[b];
  const int L = (Lraw < 0 || (int64_t)Lraw > p.stride) ? 0 : Lraw;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int pos = -1, ngram = 0;
  for (int n = p.max_ngram; n >= p.min_ngram && pos < 0; --n) {
    if (n >= L) continue;  // no earlier position can hold n tokens plus a continuation
    int32_t query[kMaxNgram];
#pragma unroll
    for (int i = 0; i < kMaxNgram; ++i) query[i] = i < n ? tok[L - n + i] : 0;
    int mine = 0x7fffffff;
    // candidate starts 0 .. L-n-1: the tokens after a match at p start at p+n <= L-1
    for (int c = threadIdx.x; c < L - n && mine == 0x7fffffff; c += kThreads) {
      bool same = true;
#pragma unroll
      for (int i = 0; i < kMaxNgram; ++i)
        if (i < n && tok[c + i] != query[i]) same = false;
      if (same) mine = c;  // this thread's candidates ascend: its first match is its earliest
    }
    mine = __reduce_min_sync(0xffffffffu, mine);
    if (lane == 0) best[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
      int m = 0x7fffffff;
      for (int w = 0; w < kThreads / 32; ++w) m = min(m, best[w]);
      found_pos = m == 0x7fffffff ? -1 : m;
    }
    __syncthreads();
    pos = found_pos;
    if (pos >= 0) ngram = n;
    __syncthreads();  // found_pos and best[] are rewritten in the next round
  }
  const int start = pos + ngram;
  const int cnt = pos >= 0 ? min(p.K, L - start) : 0;
  for (int i = threadIdx.x; i < p.K; i += kThreads) p.draft[(int64_t)b * p.K + i] = i < cnt ? tok[start + i] : -1;
  if (threadIdx.x == 0) {
    p.count[b] = cnt;
    if (p.match_pos) p.match_pos[b] = pos;
    if (p.match_ngram) p.match_ngram[b] = ngram;
  }
}

}  // namespace pld
}  // namespace fly

// Fused LM-head verification: logits = hidden x weight are formed on the 5th-gen
// tensor cores (tcgen05.mma, fp32 accumulators in tensor memory) and reduced to
// the per-row softmax statistics of Eq. 1 / Eq. 5 straight out of tensor memory;
// the logits never reach global memory.
//
// Orientation.  The vocabulary is the MMA's M dimension and the positions are
// its N dimension ("swap-AB"):  D[v, p] = sum_d weight[d, v] * hidden[p, d].
// Two CTAs on neighbouring SMs work as one pair (tcgen05 cta_group::2) on a tile
// of 256 vocabulary entries x up to 288 positions:
//   A = weight tile.  Each CTA holds ITS 128 vocabulary entries x 64 hidden dims.
//       weight is [D, V] with V contiguous, so A is MN-major; TMA lays it down as
//       two boxes of 64 entries (128 bytes) x 64 dims with the 128-byte swizzle.
//   B = hidden tile, K-major, 128-byte swizzle.  The pair shares it: each CTA
//       loads HALF of the positions of each accumulator (2 x 72 rows), the MMA
//       reads both halves.  This halves the hidden-state traffic per SM, which is
//       what bounds a one-CTA version of this kernel (the hidden tile is
//       re-fetched from L2 for every vocabulary tile).
//   D = two accumulators of 144 fp32 columns in each CTA: lane = one of the
//       CTA's 128 vocabulary entries, column = position.  Tensor memory holds
//       THREE such slots (columns 0.., 144.., 288..; 432 of 512) and the
//       accumulators of consecutive tiles rotate through them: accumulator 0 of
//       the next tile always finds a slot the epilogue is not reading, and
//       accumulator 1 takes the slot that accumulator 0 of this tile leaves,
//       which the epilogue drains first - so the tensor pipe does not wait for
//       the whole epilogue of a tile, only (at most) for its first half.
// Up to 288 positions need no padding this way (288 = 2 x 144, a legal MMA N),
// every weight tile meets all positions while it is in shared memory, and the
// weights (the only large operand) stream from HBM exactly once.
//
// Pairs are persistent: pair i walks vocabulary tiles i, i + #pairs, ...  Warp
// roles in each CTA: 0-7 epilogue (two groups of four; warp w reads the 32-lane
// quarter w % 4 of tensor memory), 8 weight producer, 9 hidden producer, 10 and
// 11 MMA issuers (leader CTA only; one per accumulator).
// "Full" barriers live in the leader: both CTAs' TMA loads report their bytes
// there.  The leader's tcgen05.commit releases a stage in both CTAs.
//
// Epilogue.  A thread that reads tensor memory owns one vocabulary entry and
// sees all positions; the reduction runs over the vocabulary.  The tile is
// therefore turned through shared memory 16 positions at a time (the two
// epilogue groups take alternate blocks, each with a buffer of its own): the
// group's four warps store their 32 x 16 blocks transposed, then thread
// (position i, vocabulary eighth e) streams the 16 logits of its eighth and
// folds them into a running (max, sum 2^t, sum 2^t t, argmax) held in registers
// for the whole kernel - the same state and the same arithmetic as the row
// reduction of the logits path, with no cross-lane traffic.  At the end the
// eight eighths are merged and the CTA writes one Partial per position; a
// later kernel folds the gridDim.x partials of every row.
//
// Every wait on a barrier is bounded: a wait that runs out records a code in
// *status, and all roles fall through to the common exit (the issuers first let
// the MMAs they already issued complete; tensor memory is released there).  No
// TMA load here is a multicast load.
#pragma once
#include <cuda.h>

#include "fly_common.cuh"
#include "mbarrier.cuh"

namespace fly {
namespace lmhead {

constexpr int kBlockV = 128;   // vocabulary entries per CTA and tile (the pair's MMA M is 256)
constexpr int kPairV = 2 * kBlockV;
constexpr int kBlockK = 64;    // hidden dims per stage: one 128-byte swizzle row of bf16
constexpr int kMmaK = 16;      // hidden dims per tcgen05.mma (bf16)
constexpr int kHalfN = 144;    // positions per accumulator (MMA N <= 256, multiple of 16)
constexpr int kMaxPos = 2 * kHalfN;
constexpr int kStages = 6;     // operand ring: one stage = one 64-dim slice of the weight tile and of the hidden tile
constexpr int kBytesW = kBlockK * kBlockV * 2;      // 16 KB per stage
constexpr int kBytesWBox = kBlockK * 64 * 2;        // one TMA box: 64 entries x 64 dims
constexpr int kBoxPos = kHalfN / 2;                 // positions per TMA box: this CTA's half of one accumulator
constexpr int kBytesHHalf = kBoxPos * kBlockK * 2;  // 9 KB
constexpr int kBytesH = 2 * kBytesHHalf;            // both accumulators
constexpr int kChunk = 16;                          // positions turned through shared memory at a time
constexpr int kChunks = kMaxPos / kChunk;           // 18 per tile, dealt alternately to the two epilogue groups
constexpr int kGroupChunks = kChunks / 2;           // 9 per group: the running states one thread holds
constexpr int kTurnRow = kBlockV + 4;               // words per position row (+4: conflict-free 128-bit reads)
constexpr int kTurnGroupBytes = kChunk * kTurnRow * 4;
constexpr int kTurnBytes = 2 * kTurnGroupBytes;     // one turning buffer per epilogue group
constexpr int kEpiWarps = 8;                        // two groups of four warps (a warp reads tensor-memory lanes 32*(warp%4)..)
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kWarpW = kEpiWarps, kWarpH = kEpiWarps + 1, kWarpMma = kEpiWarps + 2;  // producers, MMA issuers
constexpr int kThreads = (kEpiWarps + 4) * 32;
constexpr int kTmemCols = 512;
constexpr int kSlots = 3;                           // accumulator slots of kHalfN columns in tensor memory
static_assert(kSlots * kHalfN <= kTmemCols, "accumulator slots must fit in tensor memory");
constexpr int kHalfChunks = kHalfN / kChunk;        // 9 blocks of 16 positions per accumulator

constexpr int kOffW = 0;
constexpr int kOffH = kOffW + kStages * kBytesW;
constexpr int kOffTurn = kOffH + kStages * kBytesH;
constexpr int kOffBar = kOffTurn + kTurnBytes;
constexpr int kNumBars = 2 * kStages + 2 * kSlots + 1;
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kSmemBytes = kOffMisc + 32 + 1024;    // + slack to align the base to 1024 bytes
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");
static_assert(kMaxPos * 8 * 16 <= kStages * kBytesW, "final merge buffer reuses the weight ring");

constexpr int kErrTimeoutProducer = 1, kErrTimeoutMma = 2, kErrTimeoutEpilogue = 3;

struct Params {
  int R;          // positions handled by this launch (1..288)
  int n0, n1;     // MMA N of the two accumulators (multiples of 16; n1 may be 0)
  int V, D;
  int num_tiles;  // ceil(V / 256): tiles of the CTA pairs
  int num_kb;     // ceil(D / 64)
  int row0;       // first row of this launch in hidden / partials
  int w_kmajor;   // 0: weight is [D, V] (vocabulary contiguous, MN-major A); 1: weight is [V, D] (K-major A)
  float scale;    // log2(e) / temperature: logit -> base-2 exponent
  Partial* partials;  // [rows, gridDim.x]: one partial state per position and CTA
  int* status;        // 0, or the code of the first wait that ran out
};

// ---- small PTX wrappers ------------------------------------------------------

// Arrives on a barrier of the CTA with rank `cta` in the pair (cluster-scope release).
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
// shared::cluster address of `addr` (an address in this CTA's shared memory) in the CTA of rank `cta`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t cta) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta));
  return r;
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tiled TMA load into THIS CTA's shared memory; the bytes are reported to `bar`, a shared::cluster
// address that may lie in the other CTA of the pair.  No multicast.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem] over the CTA pair (M = 256: 128 rows per CTA; each CTA supplies its
// rows of A and half of B's rows from the same shared-memory offsets), bf16 inputs, fp32 accumulate.
// The shared-memory descriptors are passed as (low word, high word): only the low word (start
// address) changes from one MMA to the next.
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                         uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on `bar` (a shared::cluster address, in either CTA of the pair) once every tcgen05.mma issued
// so far by this thread has completed in both CTAs.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 16 columns of fp32: thread = lane, register i = column col0 + i.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Named barriers: 1 and 2 for the two epilogue groups (128 threads each), 3 for all epilogue threads.
__device__ __forceinline__ void group_bar(int group) { asm volatile("bar.sync %0, 128;" ::"r"(group + 1) : "memory"); }
__device__ __forceinline__ void epi_all_bar() { asm volatile("bar.sync 3, 256;" ::: "memory"); }

// ---- descriptors ---------------------------------------------------------------
// Shared-memory matrix descriptor of tcgen05.mma (64 bits).  Low word: start address and leading
// byte offset, both in 16-byte units.  High word: stride byte offset in 16-byte units, descriptor
// version 1, 128-byte swizzle.
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
  return ((addr >> 4) & 0x3fffu) | (((lbo_bytes >> 4) & 0x3fffu) << 16);
}
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);  // groups of 8 rows 1024 bytes apart
// Instruction descriptor: fp32 accumulator, bf16 A and B, A MN-major (vocabulary
// contiguous), B K-major, M = 256 (the pair), N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool a_kmajor) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_kmajor ? 0u : 1u) << 15) | (0u << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kPairV >> 4) << 24);
}

// Running statistics of one (position, vocabulary quarter) stream.
struct Stream {
  float mx, S, u;
  int idx;
};

// Folds 16 consecutive vocabulary entries x[0..15] (the first one has index v0) into st.
__device__ __forceinline__ void fold16(Stream& st, float (&x)[16], int v0, float scale) {
  float lm = kMaskFloor;
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    x[e] = max_nan_f32(x[e], kMaskFloor);  // masked entries stay finite; NaN survives and ends in S
    lm = fmaxf(lm, x[e]);
  }
  if (lm > st.mx) {  // the maximum moves: rebase the sums and record the first entry that holds it
    const float d = (st.mx - lm) * scale;
    const float sc = ex2_approx(d);
    st.u = sc * fmaf(d, st.S, st.u);
    st.S *= sc;
    st.mx = lm;
    int first = 15;
#pragma unroll
    for (int e = 15; e >= 0; --e)
      if (x[e] == lm) first = e;
    st.idx = v0 + first;
  }
  const float nr = -st.mx * scale;
  float S0 = 0.f, S1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
  for (int e = 0; e < 16; e += 2) {
    const float t0 = fmaf(x[e], scale, nr), t1 = fmaf(x[e + 1], scale, nr);
    const float e0 = ex2_approx(t0), e1 = ex2_approx(t1);
    S0 += e0;
    u0 = fmaf(e0, t0, u0);
    S1 += e1;
    u1 = fmaf(e1, t1, u1);
  }
  st.S += S0 + S1;
  st.u += u0 + u1;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
lmhead_verify_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_h,
                     const Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // swizzle atoms are 1024-byte aligned
  uint8_t* gbase = smem_raw + (base - raw);
  const uint32_t bar0 = base + kOffBar;
  // full(s), in the leader: the stage's operands of BOTH CTAs have landed (the leader's two producers
  // arrive with the expected byte counts; every TMA load of the pair reports its bytes here).
  // empty(s), in each CTA: the MMAs that read the stage have completed, the producers may refill it.
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto empty = [&](int s) { return bar0 + 8u * (kStages + s); };
  // slot_full(i), in each CTA: the accumulator in tensor-memory slot i is complete.  slot_empty(i), in the leader:
  // the epilogue threads of both CTAs have read slot i out, the next accumulator may be formed there.
  auto slot_full = [&](int i) { return bar0 + 8u * (2 * kStages + i); };
  auto slot_empty = [&](int i) { return bar0 + 8u * (2 * kStages + kSlots + i); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kStages + 2 * kSlots);  // used only on the give-up path
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(gbase + kOffMisc);  // [0] tmem base, [1], [2] go flags of the epilogue groups

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();  // 0: leader of the pair (issues the MMAs, owns the "full" barriers)
  const int pair = (int)blockIdx.x >> 1, npairs = (int)gridDim.x >> 1;

  if (threadIdx.x == 0) {
    const uint32_t issuers = p.n1 > 0 ? 2 : 1;  // one MMA-issuing thread per accumulator
    for (int s = 0; s < kStages; ++s) { mbar_init(full(s), 2); mbar_init(empty(s), issuers); }
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(slot_full(i), 1);                  // the one issuer that formed the accumulator
      mbar_init(slot_empty(i), 2 * kEpiThreads);   // the epilogue threads of both CTAs arrive on the leader's
    }
    mbar_init(drain_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {  // warp 0 of both CTAs together allocate all of tensor memory (one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kOffMisc),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // both CTAs' barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem = misc[0];

  const int my_tiles = pair < p.num_tiles ? (p.num_tiles - 1 - pair) / npairs + 1 : 0;

  if (warp == kWarpW) {
    // ---------------- weight producer: this CTA's 128 vocabulary entries ----------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      for (int t = 0; t < my_tiles && ok; ++t) {
        const int v0 = (pair + t * npairs) * kPairV + (int)rank * kBlockV;
        for (int kb = 0; kb < p.num_kb; ++kb, ++issued) {
          const int s = issued % kStages;
          const uint32_t ph = (issued / kStages) & 1;
          if (!mbar_wait(empty(s), ph ^ 1, p.status, kErrTimeoutProducer)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(full(s), 2 * kBytesW);  // both CTAs' bytes
          const uint32_t bar = map_to_cta(full(s), 0);
          const uint32_t dst = base + kOffW + s * kBytesW;
          if (p.w_kmajor) {  // [V, D]: one box of 128 entries x 64 dims, each entry's 64 dims contiguous
            tma_load_2d(dst, &map_w, kb * kBlockK, v0, bar);
          } else {           // [D, V]: two boxes of 64 entries x 64 dims, each dim's 64 entries contiguous
            tma_load_2d(dst, &map_w, v0, kb * kBlockK, bar);
            tma_load_2d(dst + kBytesWBox, &map_w, v0 + 64, kb * kBlockK, bar);
          }
        }
      }
    }
  } else if (warp == kWarpH) {
    // ---------------- hidden-state producer: this CTA's half of each accumulator's positions ----------------
    if (lane == 0) {
      int issued = 0;
      bool ok = true;
      const uint32_t bytes = p.n1 > 0 ? kBytesH : kBytesHHalf;
      const int y0 = p.row0 + (int)rank * (p.n0 / 2);
      const int y1 = p.row0 + kHalfN + (int)rank * (p.n1 / 2);
      for (int t = 0; t < my_tiles && ok; ++t) {
        for (int kb = 0; kb < p.num_kb; ++kb, ++issued) {
          const int s = issued % kStages;
          const uint32_t ph = (issued / kStages) & 1;
          if (!mbar_wait(empty(s), ph ^ 1, p.status, kErrTimeoutProducer)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(full(s), 2 * bytes);
          const uint32_t bar = map_to_cta(full(s), 0);
          const uint32_t dst = base + kOffH + s * kBytesH;
          tma_load_2d(dst, &map_h, kb * kBlockK, y0, bar);
          if (p.n1 > 0) tma_load_2d(dst + kBytesHHalf, &map_h, kb * kBlockK, y1, bar);
        }
      }
    }
  } else if (warp >= kWarpMma) {
    // ---------------- MMA issuers (leader CTA): warp 6 feeds accumulator 0, warp 7 accumulator 1 ----------------
    // One thread cannot issue MMAs, commits and barrier waits fast enough to keep the tensor pipe
    // busy with two 144-column MMAs per 16 hidden dims, so each accumulator has an issuer of its own.
    const int half = warp - kWarpMma;
    if (lane == 0 && rank == 0 && (half == 0 || p.n1 > 0)) {
      const uint32_t idesc = instr_desc(half == 0 ? p.n0 : p.n1, p.w_kmajor != 0);
      const int nh = p.n1 > 0 ? 2 : 1;  // accumulators per tile
      // Everything that changes from one MMA to the next is a 32-bit add: this thread has to issue one
      // MMA every ~70 cycles, so the loop is kept to a few instructions per MMA.
      // A, MN-major: 64-entry chunks lie kBytesWBox apart (leading offset), groups of 8 hidden dims
      // 1024 bytes apart (stride offset); 16 hidden dims further = 16 rows of 128 bytes.
      // B, K-major: groups of 8 positions 1024 bytes apart; 16 hidden dims further = 32 bytes.
      // With the weight stored [V, D] A is K-major like B: 128 rows of 128 bytes, 16 dims further = 32 bytes.
      const uint32_t a_lo0 = p.w_kmajor ? desc_lo(base + kOffW, 16) : desc_lo(base + kOffW, kBytesWBox);
      const uint32_t a_step = p.w_kmajor ? (uint32_t)((kMmaK * 2) >> 4) : (uint32_t)((kMmaK * 128) >> 4);
      const uint32_t b_lo0 = desc_lo(base + kOffH + half * kBytesHHalf, 16);
      const uint32_t peer_delta = map_to_cta(bar0, 1) - bar0;  // same offset in the partner's shared memory
      int st = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int t = 0; t < my_tiles && ok; ++t) {
        // this accumulator's slot: the (t * nh + half)-th use of the rotation; the epilogue must have read out
        // what the slot held three uses ago
        const int use = t * nh + half;
        const int slot = use % kSlots;
        const uint32_t d_tmem = tmem + (uint32_t)(slot * kHalfN);
        if (!mbar_wait(slot_empty(slot), ((use / kSlots) & 1) ^ 1, p.status, kErrTimeoutMma)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < p.num_kb; ++kb) {
          // TMA-written operands need no tcgen05 fence: the barrier wait orders them before the MMAs
          if (!mbar_wait(full(st), ph, p.status, kErrTimeoutMma)) { ok = false; break; }
          const uint32_t a_lo = a_lo0 + (uint32_t)st * (kBytesW >> 4);
          const uint32_t b_lo = b_lo0 + (uint32_t)st * (kBytesH >> 4);
#pragma unroll
          for (int ks = 0; ks < kBlockK / kMmaK; ++ks) {
            const uint32_t acc = ks == 0 ? (uint32_t)(kb != 0) : 1u;
            mma_bf16(d_tmem, a_lo + ks * a_step, b_lo + ks * ((kMmaK * 2) >> 4), kDescHi, idesc, acc);
          }
          // the stage may be refilled, in both CTAs, once these MMAs have read it
          const uint32_t eb = empty(st);
          mma_commit(eb);
          mma_commit(eb + peer_delta);
          if (++st == kStages) { st = 0; ph ^= 1; }
        }
        if (ok) {
          mma_commit(slot_full(slot));
          mma_commit(slot_full(slot) + peer_delta);
        }
      }
      if (!ok) {
        // Give-up path: MMAs issued before the failed wait may still be reading shared memory and writing
        // tensor memory.  One more commit to a barrier of its own, and a (bounded) wait on it, lets them
        // finish before the common exit hands both back.
        mma_commit(drain_bar);
        mbar_wait_quiet(drain_bar, 0, 2000000ull);
      }
    }
  } else {
    // ---------------- epilogue: warps 0..7 = two groups of four warps ----------------
    // Group g turns the 16-position blocks c = g, g+2, ... of every tile.  Inside a group, warp q
    // reads tensor-memory lanes 32q.. (its quarter of the CTA's vocabulary entries) and stores them
    // transposed; then thread (position i = tid & 15, vocabulary eighth e = tid >> 4) folds its 16 logits.
    const int group = warp >> 2, q = warp & 3;
    const int gtid = threadIdx.x & 127;              // thread index inside the group
    const int pos_i = gtid & 15, eighth = gtid >> 4;
    Stream st[kGroupChunks];
#pragma unroll
    for (int k = 0; k < kGroupChunks; ++k) { st[k].mx = kMaskFloor; st[k].S = 0.f; st[k].u = 0.f; st[k].idx = kIdxNone; }
    float* turn = reinterpret_cast<float*>(gbase + kOffTurn + group * kTurnGroupBytes);
    const int nchunks = (p.R + kChunk - 1) / kChunk;                 // blocks of this launch
    const int my_chunks = nchunks > group ? (nchunks - group + 1) / 2 : 0;  // ... that this group turns
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const int nh = p.n1 > 0 ? 2 : 1;
    // the last block of each accumulator that this group turns (-1: none): after reading it the thread hands the
    // accumulator's slot back
    int last0 = -1, last1 = -1;
    for (int k = 0; k < my_chunks; ++k) {
      if (2 * k + group < kHalfChunks) last0 = k;
      else last1 = k;
    }
    for (int t = 0; t < my_tiles; ++t) {
      const int use0 = t * nh, use1 = t * nh + 1;
      const int slot0 = use0 % kSlots, slot1 = use1 % kSlots;
      if (gtid == 0) {
        bool okw = mbar_wait(slot_full(slot0), (use0 / kSlots) & 1, p.status, kErrTimeoutEpilogue);
        if (okw && nh == 2) okw = mbar_wait(slot_full(slot1), (use1 / kSlots) & 1, p.status, kErrTimeoutEpilogue);
        misc[1 + group] = okw ? 1u : 0u;
      }
      group_bar(group);
      const bool go = misc[1 + group] != 0;  // one thread per group waits, the group takes the same decision
      if (!go) break;
      tc_fence_after();
      const int v0 = (pair + t * npairs) * kPairV + (int)rank * kBlockV + eighth * 16;
      const int limit = p.V - v0;  // entries of this eighth that exist
      // an accumulator of which this group turns no block is handed back at once
      if (last0 < 0) { tc_fence_before(); mbar_arrive_remote(map_to_cta(slot_empty(slot0), 0)); }
      if (nh == 2 && last1 < 0) { tc_fence_before(); mbar_arrive_remote(map_to_cta(slot_empty(slot1), 0)); }
#pragma unroll
      for (int k = 0; k < kGroupChunks; ++k) {
        if (k < my_chunks) {
          const int c = 2 * k + group;
          const int h = c / kHalfChunks;  // which accumulator the block belongs to
          uint32_t r[16];
          tmem_ld16(tmem + lane_base + (uint32_t)((h ? slot1 : slot0) * kHalfN + (c - h * kHalfChunks) * kChunk), r);
          if (k == (h ? last1 : last0)) {  // last read of this accumulator by this thread: hand its slot back
            tc_fence_before();
            mbar_arrive_remote(map_to_cta(slot_empty(h ? slot1 : slot0), 0));
          }
          group_bar(group);  // the group is done reading the previous block
#pragma unroll
          for (int i = 0; i < 16; ++i) turn[i * kTurnRow + q * 32 + lane] = __uint_as_float(r[i]);
          group_bar(group);
          float x[16];
          const float4* src = reinterpret_cast<const float4*>(turn + pos_i * kTurnRow + eighth * 16);
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const float4 v = src[jj];
            x[4 * jj] = v.x; x[4 * jj + 1] = v.y; x[4 * jj + 2] = v.z; x[4 * jj + 3] = v.w;
          }
          if (limit < 16) {  // ragged vocabulary: entries past V do not exist
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (e >= limit) x[e] = kMaskFloor;
          }
          fold16(st[k], x, v0, p.scale);
        }
      }
    }
    // Merge the eight vocabulary eighths of every position and write the CTA's partial state.
    // The weight ring is free by now: every MMA that read it has completed (slot_full of the last tile).
    epi_all_bar();
    Partial* buf = reinterpret_cast<Partial*>(gbase + kOffW);
#pragma unroll
    for (int k = 0; k < kGroupChunks; ++k) {
      Partial pq;
      pq.mx = st[k].mx; pq.S = st[k].S; pq.u = st[k].u; pq.idx = st[k].idx;
      buf[((2 * k + group) * kChunk + pos_i) * 8 + eighth] = pq;
    }
    epi_all_bar();
    for (int pos = threadIdx.x; pos < p.R; pos += kEpiThreads) {
      Partial a = buf[pos * 8];
#pragma unroll
      for (int e = 1; e < 8; ++e) merge_partial(a, buf[pos * 8 + e], p.scale);
      p.partials[(int64_t)(p.row0 + pos) * gridDim.x + blockIdx.x] = a;
    }
  }

  // Common exit.  After a failed wait give stragglers (TMA copies still in flight towards this
  // CTA's shared memory) time to land before the shared memory is handed back.
  if (*(volatile int*)p.status != 0) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 2000000ull) {}
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();  // neither CTA leaves while its partner may still signal its barriers or read its operands
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// Exercises the bounded wait without any fault: one thread waits on a barrier that nothing will
// ever complete; after limit_ns the wait gives up and records `code`.
constexpr int kErrSelfTest = 9;
__global__ void wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t b = smem_u32(&bar);
  mbar_init(b, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  mbar_wait(b, 0, status, kErrSelfTest, limit_ns);
}

}  // namespace lmhead
}  // namespace fly

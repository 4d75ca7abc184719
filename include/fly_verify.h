/*
 * fly_verify.h - C ABI of the FLy loose-verification step for NVIDIA B200 (sm_100a).
 *
 * One call verifies one speculative-decoding round for a batch of sequences:
 * for each of the K+1 target-model logit rows of a sequence it computes the
 * softmax entropy and the greedy token (Eq. 1, Eq. 5), compares the greedy
 * tokens with the K draft tokens (Eq. 2), applies the entropy gate (Eq. 6) and
 * the deferred-window rule (Eq. 8 - Eq. 11; Algorithm 1, steps 3 and 4) and
 * writes the accepted-token count and the tokens to append.
 *
 * Conventions
 *   - Every pointer marked "dev" is device memory of the handle's device, owned
 *     by the caller; the library never frees or keeps it.  Pointers marked
 *     "host" are host memory.
 *   - Rows: sequence b, position i (1-based, 1..K+1) is row b*(K+1) + (i-1).
 *     Position K+1 is the bonus position.
 *   - fly_verify_run is asynchronous on the given CUDA stream, allocates
 *     nothing and never synchronises the host with the device.
 *   - A handle owns one set of scratch buffers: steps issued through one handle
 *     must run one after the other on the GPU (keep a handle on one stream at a
 *     time) and the host calls on it must not overlap (one host thread at a
 *     time).  Use one handle per stream.
 *   - No function throws, aborts or traps.  Misuse that the host can see is
 *     reported by the return code before anything is launched; conditions that
 *     depend on device data (non-finite logits, draft ids out of range) are
 *     reported per row in row_flags.
 */
#ifndef FLY_VERIFY_H_
#define FLY_VERIFY_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fly_verify fly_verify_t; /* opaque; owns scratch memory only */

typedef enum {
  FLY_OK = 0,
  FLY_ERR_INVALID_ARG = 1, /* null pointer, size out of range, inconsistent arguments */
  FLY_ERR_UNSUPPORTED = 2, /* a valid request this build cannot serve (alignment, W > K in carry mode, ...) */
  FLY_ERR_CUDA = 3,        /* a CUDA runtime call failed; see fly_verify_last_cuda_error */
  FLY_ERR_TIMEOUT = 4,     /* a bounded device-side wait ran out (fused path) */
  FLY_ERR_TOO_LARGE = 5    /* fly_verify_run_static only: the step does not fit the built-in scratch area */
} fly_status_t;

typedef enum { FLY_F32 = 0, FLY_BF16 = 1 } fly_dtype_t;

/* Unit of the gate threshold theta.  The paper thresholds the normalised
 * entropy h = H / log|V| in [0,1] (Eq. 5, Eq. 6).  NATS compares H (natural
 * log) with theta directly; NORMALIZED compares H with theta * log(vocab). */
typedef enum { FLY_THETA_NATS = 0, FLY_THETA_NORMALIZED = 1 } fly_theta_unit_t;

/* What happens to a Defer mismatch j whose window j+1..j+W does not fit in the
 * round (j + W > K).  REJECT is the paper's rule (the paragraph after Eq. 9):
 * the mismatch is rejected at once and no state crosses rounds.  CARRY is an
 * extension: if positions j+1..K hold no mismatch the token is kept
 * provisionally and the remaining j+W-K window slots are checked against the
 * first draft positions of the next round; a mismatch there revokes it. */
typedef enum { FLY_BOUNDARY_REJECT = 0, FLY_BOUNDARY_CARRY = 1 } fly_boundary_t;

/* Deferred state of one sequence between rounds (CARRY only).
 * pending      window slots still open at the start of the next round (0: none)
 * rollback_len tokens appended since and including the provisionally kept mismatch
 * correction   the target's own token at that mismatch
 * The zero state is {0, 0, -1}. */
typedef struct {
  int32_t pending;
  int32_t rollback_len;
  int32_t correction;
} fly_state_t;

typedef struct {
  int32_t device;           /* CUDA device ordinal */
  int32_t max_batch;        /* largest B of any run, >= 1 */
  int32_t max_k;            /* largest K of any run, 1..63 */
  int32_t vocab;            /* |V| >= 1: row length of the logits */
  fly_dtype_t logits_dtype; /* storage type of the logits */
  int32_t hidden;           /* 0: logits path only.  > 0: hidden size of the fused LM-head path */
} fly_verify_config_t;

/* Creates a handle and its scratch memory (per-row partial states for rows
 * that are split over several thread blocks).  host pointers.  On failure
 * *out is NULL. */
fly_status_t fly_verify_create(const fly_verify_config_t* config, fly_verify_t** out);

/* Frees the scratch memory and the handle.  NULL is accepted. */
fly_status_t fly_verify_destroy(fly_verify_t* handle);

typedef struct {
  int32_t B; /* sequences, 1..max_batch */
  int32_t K; /* draft tokens per sequence, 1..max_k */

  /* Logits path: dev [B, K+1, V] of logits_dtype, V contiguous, consecutive rows
   * row_stride elements apart (row_stride >= V; 0 means V). */
  const void* logits;
  int64_t row_stride;

  /* Fused LM-head path (logits == NULL; the handle was created with hidden > 0):
   * the logits are hidden x weight - the last linear layer of the target forward
   * pass that yields l_1..l_{K+1} (Section 2.1) - formed in fp32 on the tensor
   * cores and never stored.
   * hidden: dev [B*(K+1), hidden] bf16 row-major, 16-byte aligned.
   * weight: dev [hidden, V] bf16 row-major (V contiguous), 16-byte aligned
   *         (or [V, hidden] with FLY_OPT_WEIGHT_LAYOUT = 1).
   * hidden and V must be multiples of 8 (fly_verify_create checks).  Positions
   * are processed 288 at a time; each block of 288 streams the weight once. */
  const void* hidden;
  const void* weight;

  const int32_t* draft; /* dev [B, K] draft tokens yhat_1..yhat_K */

  double theta;                /* gate threshold (Eq. 6); +inf gives exact-match acceptance (Eq. 3) */
  fly_theta_unit_t theta_unit;
  int32_t W;                   /* window length >= 0 (Eq. 8) */
  fly_boundary_t boundary;

  const fly_state_t* state_in; /* dev [B] or NULL (= zero state); CARRY only */
  fly_state_t* state_out;      /* dev [B]; required for CARRY, optional for REJECT (zero state written).
                                  May alias state_in. */

  int32_t* accept_len;    /* dev [B]: s in 1..K+1, tokens to append this round (Eq. 11) */
  int32_t* rollback;      /* dev [B] or NULL: tokens to remove BEFORE appending (non-zero only when a
                             carried deferral is revoked) */
  int32_t* out_tokens;    /* dev [B, K+1]: first s entries valid, the rest -1 (Algorithm 1's concat lines) */
  int32_t* target_argmax; /* dev [B, K+1] or NULL: y_i of Eq. 1, lowest index among equal maxima */
  float* entropy;         /* dev [B, K+1] or NULL: H_i in nats (numerator of Eq. 5) */
  uint32_t* row_flags;    /* dev [B, K+1] or NULL: bit 0 non-finite logit (NaN, +inf, or no finite entry);
                             bit 1 draft id outside [0, V) (treated as a mismatch);
                             bit 2 caller-supplied target token outside [0, V) (mismatch, never deferred);
                             bit 3 (on position 1 only) the carried state read from state_in is not one this
                                   library writes (pending outside [0, K], negative rollback_len, or a pending
                                   window whose correction token is outside [0, V)): it is ignored, i.e. the
                                   round is verified from the zero state;
                             bit 4 fused path only: a bounded wait of the GEMM kernel ran out during this step
                                   (see fly_verify_device_status); set on every row, every position counts as a
                                   mismatch that is never deferred, so accept_len is 1 and nothing drafted is kept */

  /* Optional (NULL = greedy): dev [B, K+1] tokens y_1..y_{K+1} that the caller drew from the target
   * distributions, e.g. by sampling at temperature 1.  The paper's method text defines y_i only as the
   * argmax (Eq. 1) although it reports temperature-1 results, so this is a hook, not the paper's rule:
   * the given tokens replace the argmax in the match indicator (Eq. 2) and in the emitted tokens;
   * the entropy gate still uses the entropy of the logits (at `temperature`).  target_argmax still reports
   * the argmax. */
  const int32_t* target_tokens;

  /* Temperature T of the target distribution: the entropy of Eq. 5 is taken of softmax(l / T), the
   * distribution a caller that samples at temperature T draws from (the paper reports temperature-1
   * results next to the greedy ones).  0 means 1 (the logits as they are); otherwise 1e-6 <= T <= 1e6.
   * 1/T is folded into the constant that turns a logit into a base-2 exponent, so it costs nothing.  The
   * greedy token (Eq. 1) does not depend on T. */
  double temperature;

  /* Launch ordering of the logits path.  The row reduction is always launched so that it may be
   * scheduled while the previous kernel in the stream drains (programmatic dependent launch).
   * 0 (default): plain stream order.  The kernel waits for the previous kernel to complete before its
   *    first read; only its launch latency is hidden.  Always correct.
   * 1: the caller guarantees that the logits and draft tokens of this step were complete BEFORE the
   *    previous kernel in the stream was launched (e.g. a queue of steps over inputs that are already in
   *    memory).  The kernel then starts READING at once, next to the draining previous kernel, and waits
   *    only before its first write.  (state_in is read after that wait: it may be the previous step's
   *    state_out.)  Wrong results if the guarantee does not hold - in a decode loop, where the previous
   *    kernel produces this step's logits, leave it 0. */
  int32_t inputs_ready;
} fly_verify_args_t;

/* Runs one verification step on `cuda_stream` (a cudaStream_t; NULL = default
 * stream).  Exactly one of args->logits / (args->hidden, args->weight) is set.
 * Returns FLY_OK once the work is enqueued. */
fly_status_t fly_verify_run(fly_verify_t* handle, const fly_verify_args_t* args, void* cuda_stream);

/* Convenience for callers that hold HOST buffers: the same step with every
 * pointer in args a host pointer (state_in/state_out included).  Inputs are
 * copied to device staging buffers owned by the handle, the step runs, results
 * are copied back and the stream is synchronised before returning.  Host
 * buffers should be page-locked for full copy bandwidth.  On the fused path
 * hidden is a host pointer; weight (a model parameter, not a per-step input)
 * remains a DEVICE pointer. */
fly_status_t fly_verify_run_host(fly_verify_t* handle, const fly_verify_args_t* args, void* cuda_stream);

/* Vocabulary-parallel targets.  The paper runs its 405B target "distributed across four GPUs"
 * (Section 3, implementation details); with a tensor-parallel LM head every GPU holds the logits of
 * one slice of the vocabulary only.  Eq. 1 and Eq. 5 then split into a per-slice reduction and a
 * merge: for a slice with maximum m_k, S_k = sum 2^(z - r_k) and u_k = sum 2^(z - r_k)(z - r_k)
 * (z = logit * log2 e / T, r_k = m_k * log2 e / T, T = the temperature, which every rank and the merging
 * call must pass alike; 0 = 1), the whole row has m = max m_k,
 * S = sum_k 2^(r_k - r) S_k, u = sum_k 2^(r_k - r)(u_k + (r_k - r) S_k), entropy
 * H = ln2 (log2 S - u / S), and the greedy token is the index of the largest m_k (lowest index on
 * ties).  One state per row and rank (16 bytes) is all that has to cross the interconnect.
 *
 * fly_verify_reduce_shard    on every rank: reduces this rank's logits [rows, vocab] (vocab = the
 *                            handle's vocab = the slice width; row_stride elements between rows, 0 = vocab)
 *                            to partial_out[rows].  vocab_offset = global id of the slice's first token.
 * (all-gather partial_out over the ranks: [world, rows] states, e.g. with NCCL)
 * fly_verify_run_partials    on every rank (or one): merges the gathered states and applies the gate and
 *                            the deferred window exactly as fly_verify_run does.  args: as for
 *                            fly_verify_run with logits, hidden and weight NULL; total_vocab = |V| (used for
 *                            the draft-id range check and for a NORMALIZED threshold).
 * All pointers dev.  Both calls are asynchronous on `cuda_stream` and allocate nothing. */
typedef struct {
  float max_logit;  /* m_k; a slice with no finite entry reports a value <= -999424 */
  float sum_exp2;   /* S_k */
  float sum_exp2_t; /* u_k */
  int32_t argmax;   /* global token id of the first entry equal to m_k */
} fly_partial_t;
fly_status_t fly_verify_reduce_shard(fly_verify_t* handle, int32_t rows, const void* logits, int64_t row_stride,
                                     int32_t vocab_offset, double temperature, fly_partial_t* partial_out,
                                     void* cuda_stream);
fly_status_t fly_verify_run_partials(fly_verify_t* handle, const fly_verify_args_t* args, const fly_partial_t* partials,
                                     int32_t world, int32_t total_vocab, void* cuda_stream);

/* Prompt-lookup drafting: the step BEFORE verification.  Section 2.3 (multi-level acceleration) speeds
 * the drafter up with prompt lookup decoding, "a simple n-gram retrieval method"; the paper gives no
 * parameters, so the rule is the cited method's: the sequence's last n tokens are searched in its
 * own earlier tokens, n from max_ngram down to min_ngram; at the first n with a match the EARLIEST
 * match position p wins and the tokens that followed it, tokens[p+n .. p+n+K) cut at the sequence end,
 * are proposed.
 *   tokens   dev [B, stride] int32, sequence b holds lengths[b] <= stride tokens (a length outside
 *            [0, stride] is treated as 0: nothing is proposed, nothing outside the row is read)
 *   draft    dev [B, K]: count[b] proposed tokens, then -1      count  dev [B] (0: no match)
 *   match_pos / match_ngram   dev [B] or NULL: p (-1: none) and n (0: none)
 * 1 <= min_ngram <= max_ngram <= 8.  No handle, no scratch; asynchronous on `cuda_stream`. */
fly_status_t fly_pld_draft(int32_t device, int32_t B, const int32_t* tokens, int64_t stride, const int32_t* lengths,
                           int32_t max_ngram, int32_t min_ngram, int32_t K, int32_t* draft, int32_t* count,
                           int32_t* match_pos, int32_t* match_ngram, void* cuda_stream);

/* The paper has no counterpart of this entry point; it exists for callers that
 * must not allocate device memory.
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they
 * verify: an inference server that has handed the whole device to its own
 * memory pool, a plugin that runs inside another framework's execution
 * callback, code that sits in a latency-critical loop where an allocation (an
 * implicit device synchronisation) is not acceptable.  fly_verify_create
 * allocates the scratch memory of a handle, so it is closed to them.  This
 * function runs the same logits-path step (same kernels, same results) with NO
 * handle: the per-piece partial states and the per-sequence arrival counters
 * live in a fixed array that is part of the library image itself
 * (FLY_STATIC_SCRATCH_BYTES of device memory on every GPU on which the library
 * is loaded, held until the process exits).  It calls no cudaMalloc, cudaFree
 * or other allocating routine.
 *
 *   device, vocab, logits_dtype   what fly_verify_config_t would carry
 *   args                          as for fly_verify_run, device pointers, logits path only (hidden and
 *                                 weight must be NULL); inputs and outputs are still the caller's
 *
 * Limits: B <= FLY_STATIC_MAX_BATCH, K <= 63 and B*(K+1) <= FLY_STATIC_MAX_PIECES.  Rows are cut into
 * pieces as usual, but the partial-state slots of all rows together never exceed FLY_STATIC_MAX_PIECES.
 * A step beyond the limits returns FLY_ERR_TOO_LARGE and launches nothing.
 *
 * The first call on each device looks up the device address of the built-in
 * array (which also makes the CUDA runtime load the library's device code).
 * Make that first call outside any stream capture; later calls only enqueue
 * work on `cuda_stream` (one memset of the B arrival counters, one kernel).
 *
 * All calls on a device share the one array, and it keeps whatever the last
 * call left there.  The counters are cleared on the stream at the start of
 * every call and the partial states are fully rewritten before they are read,
 * so stale contents never leak into a result.  But two calls whose work
 * overlaps on the GPU (different streams, or several host threads) write the same
 * scratch and corrupt each other: serialise them, e.g. keep them on one stream. */
#define FLY_STATIC_MAX_BATCH 1024
#define FLY_STATIC_MAX_PIECES 16384
#define FLY_STATIC_SCRATCH_BYTES (FLY_STATIC_MAX_BATCH * 4 + FLY_STATIC_MAX_PIECES * 16) /* 260 KiB */
fly_status_t fly_verify_run_static(int32_t device, int32_t vocab, fly_dtype_t logits_dtype,
                                   const fly_verify_args_t* args, void* cuda_stream);

/* Options of a handle (fly_verify_set_option).  None of them changes results
 * beyond fp32 rounding order.
 *
 * FLY_OPT_SPLITS          How the row reduction cuts rows into thread-block ranges.  0 (default): every row is cut
 *                         into the same number of whole pieces (at least 16 KB each) - in plain stream order the
 *                         count that keeps the grid on the device at once with the least work on the busiest SM,
 *                         with inputs_ready few large pieces, so that consecutive steps overlap many deep; where
 *                         whole pieces would leave most of the last wave of blocks empty, the rows are laid end
 *                         to end and that range is cut evenly instead (a block may then cover the end of one row
 *                         and the start of the next).
 *                         s > 0: every row is cut into exactly s pieces (1..32), one thread block each (for
 *                         tests and experiments).
 * FLY_OPT_SCAN_MODE       0 (default): the acceptance scan runs as the tail of the row-reduction
 *                         kernel (the block that completes a sequence's rows verifies it; one launch
 *                         per step).  1: it runs as a kernel of its own (two launches per step).
 * FLY_OPT_WEIGHT_LAYOUT   fused path only.  0 (default): weight is [hidden, V] row-major (V contiguous).
 *                         1: weight is [V, hidden] row-major (hidden contiguous), the layout in which
 *                         linear layers are usually stored. */
typedef enum {
  FLY_OPT_SPLITS = 0,
  FLY_OPT_SCAN_MODE = 1,
  FLY_OPT_WEIGHT_LAYOUT = 3
} fly_option_t;
fly_status_t fly_verify_set_option(fly_verify_t* handle, fly_option_t option, int32_t value);

/* The fused path's kernel waits on hardware barriers (TMA arrival, tensor-core
 * completion); every such wait is bounded.  If one runs out, the kernel records
 * it and returns without hanging (its outputs are then undefined).  This call
 * synchronises `cuda_stream` and returns FLY_ERR_TIMEOUT if that happened since
 * the last call (the record is cleared), else FLY_OK.  While a record is
 * pending, further fused steps give up early, and every step run in that state
 * marks all of its rows with row_flags bit 4, so the failure is also visible in
 * stream order without a host synchronisation.  Logits-path kernels have no waits. */
fly_status_t fly_verify_device_status(fly_verify_t* handle, void* cuda_stream);

/* Self-test of that mechanism, safe to run anywhere: enqueues a one-thread kernel that waits, with a
 * 2 ms limit, on a barrier nothing will complete.  The wait gives up, the kernel returns normally, and the
 * next fly_verify_device_status reports FLY_ERR_TIMEOUT.  Nothing faults or hangs. */
fly_status_t fly_verify_selftest_wait(fly_verify_t* handle, void* cuda_stream);

/* Introspection, host only (no CUDA call): the launch geometry the logits path chooses for `rows` rows of
 * `vocab` logits of `dtype` on a device with sm_count SMs.  vector_path = 1 if base, row stride and row length
 * allow 16-byte loads (a unit is then a 16-byte segment, else one logit).  forced_pieces as FLY_OPT_SPLITS.
 *   grid             thread blocks
 *   units_per_block  block b reduces the flat unit range [b * units_per_block, (b + 1) * units_per_block)
 *   units_per_row    whole units in a row
 *   row_span         units a row takes in that flat range (>= units_per_row; equal when rows are packed
 *                    end to end, a multiple of units_per_block when rows are cut into whole pieces)
 *   slots            partial-state slots reserved per row (>= the pieces of any row)
 * Returns FLY_ERR_INVALID_ARG for sizes out of range. */
typedef struct {
  int32_t grid;
  int32_t slots;
  int64_t units_per_block;
  int64_t units_per_row;
  int64_t row_span;
} fly_plan_t;
fly_status_t fly_verify_plan(int32_t sm_count, int64_t rows, int32_t vocab, fly_dtype_t dtype, int32_t vector_path,
                             int32_t inputs_ready, int32_t forced_pieces, fly_plan_t* out);

/* Number of kernels the last fly_verify_run enqueued (for accounting). */
int32_t fly_verify_last_launch_count(const fly_verify_t* handle);

/* cudaError_t value of the last failed CUDA call on this handle (0 if none). */
int32_t fly_verify_last_cuda_error(const fly_verify_t* handle);

const char* fly_status_string(fly_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* FLY_VERIFY_H_ */

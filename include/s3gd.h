/*
 * s3gd.h -- C ABI of the S3GD-MV compression / aggregation / update step for
 * one NVIDIA B200 (sm_100a).
 *
 * The operations are those of Park & Lee, "Sparse-SignSGD with Majority Vote
 * for Communication-Efficient Distributed Learning" (arXiv 2302.07475):
 * M workers each hold a gradient of length d (the paper's N); each sends the
 * signs of its K largest-magnitude entries (TopKSign, Section 2.1 Eq. (3)-(4)),
 * the server takes the sign of the summed votes (Section 2.2 "Majority vote",
 * Algorithm 1) and every worker moves x by -lr times that sign vector
 * (Section 2.2 Eq. (7)).  Here the M workers are the rows of one gradient
 * buffer in device memory and the "network" is device memory.
 *
 * Conventions shared by every call
 * --------------------------------
 *  - "dev" pointers are device pointers valid on the current CUDA device;
 *    "host" means ordinary host memory.  The library never allocates, frees or
 *    retains a pointer.  Every buffer, including the workspace, is the caller's.
 *  - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *    the default stream).  No call synchronises except s3gd_device_status(),
 *    s3gd_last_device_status() and s3gd_profile_end().  Stream order is kept: some kernels are
 *    launched so that their blocks may be scheduled while the previous kernel on the stream
 *    (the caller's included) is still draining, but they touch no memory before it has completed.
 *  - Magnitude order is the unsigned order of the fp32 bit pattern with the sign
 *    bit cleared.  Denormals are not flushed; NaN and Inf order by bit pattern.
 *  - Exactly K entries are kept per worker; equal magnitudes go to the lower
 *    index.  A kept entry votes with its IEEE sign bit (+0 votes +1, -0 votes -1).
 *  - Indices are 0-based uint32 and ascending within a worker.  Sign bit j of a
 *    worker belongs to its j-th index: word j/32, bit j%32 (LSB first),
 *    1 = negative; unused bits of the last word are 0.
 *  - Return value: S3GD_OK, or an argument / workspace error detected on the host
 *    BEFORE anything is enqueued (outputs untouched).  S3GD_ERR_CUDA reports a failed
 *    CUDA runtime call and may come after part of the call's work was enqueued: the
 *    outputs are then undefined.  Conditions only the device can see are recorded
 *    in the workspace and read back with s3gd_device_status().
 *  - Limits: 1 <= M <= 65535 workers, 1 <= d < 2^32 coordinates, 0 <= K <= d.
 *  - Threads: calls on different workspaces may be made from different host threads
 *    (the only shared host state is a set of per-device caches that are written once).
 *    Calls that share a workspace must be ordered by the caller.  Not thread-safe:
 *    the s3gd_profile_* calls (one session per process; do not open or close one while
 *    another thread is inside a step) and s3gd_majority_vote_noalloc (one built-in
 *    scratch array per device).
 */
#ifndef S3GD_H_
#define S3GD_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define S3GD_API __attribute__((visibility("default")))
#else
#define S3GD_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum s3gd_status {
  S3GD_OK = 0,
  S3GD_ERR_INVALID_ARG = 1, /* NULL pointer, M <= 0, M > 65535, d == 0, d >= 2^32, K > d, bad alignment */
  S3GD_ERR_WORKSPACE = 2,   /* workspace NULL, smaller than s3gd_workspace_bytes(), or not 256-byte aligned */
  S3GD_ERR_CUDA = 3,        /* a CUDA runtime call failed (launch error, wrong device, no room to load the
                               library's GPU code, ...); outputs may be partly written */
  S3GD_ERR_INDEX_RANGE = 4, /* device: an index >= d was given to s3gd_majority_vote (skipped) */
  S3GD_ERR_INTERNAL = 5,    /* device: a selection did not produce exactly K entries */
  S3GD_ERR_TOO_LARGE = 6    /* s3gd_majority_vote_noalloc: d exceeds s3gd_noalloc_max_d() */
} s3gd_status;

/* Human-readable name of a status code.  Host.  Never NULL. */
S3GD_API const char* s3gd_status_string(s3gd_status st);

/*
 * Bytes of device workspace that the calls below need for (M, d, K).  Host, pure.
 * A workspace sized for (M, d, K) is only guaranteed to serve calls with exactly
 * these three values.  Returns 0 for invalid arguments.  The workspace must be
 * 256-byte aligned.  Its contents need not be initialised and are not preserved.
 */
S3GD_API size_t s3gd_workspace_bytes(int M, uint64_t d, uint64_t K);

/*
 * TopKSign of every worker's gradient in transmitted form
 * (Section 2.1, Eq. (3)-(4); Section 2.2 "Gradient compression").
 *
 *  grads        dev, const  [M x d] fp32 row-major (row m = worker m), 4-byte aligned
 *  out_idx      dev         [M x K] uint32, ascending per row
 *  out_signbits dev         [M x ceil(K/32)] uint32
 *  ws, ws_bytes dev         workspace, >= s3gd_workspace_bytes(M, d, K)
 *
 * K == 0 is valid and writes nothing.  K == d keeps everything.
 */
S3GD_API s3gd_status s3gd_topk_sign(const float* grads, int M, uint64_t d, uint64_t K,
                           uint32_t* out_idx, uint32_t* out_signbits,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * Majority vote at the server (Section 2.2 "Majority vote"; Algorithm 1):
 * out_vote[n] = sgn( sum over workers and their entries j with idx == n of
 * (1 - 2 * signbit_j) ), so a coordinate nobody sent, or an exact tie, gets 0.
 *
 *  idx       dev, const  [M x K] uint32 (any order; repeated indices add up;
 *                        an index >= d is skipped and S3GD_ERR_INDEX_RANGE is recorded)
 *  signbits  dev, const  [M x ceil(K/32)] uint32
 *  out_vote  dev         [d] int8 in {-1, 0, +1}
 *  ws        dev         workspace, >= s3gd_workspace_bytes(M, d, K); holds the int32 counters
 */
S3GD_API s3gd_status s3gd_majority_vote(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K,
                               uint64_t d, int8_t* out_vote,
                               void* ws, size_t ws_bytes, void* stream);

/*
 * Model update (Section 2.2, Eq. (7)): x[n] <- fl32(x[n] - lr * vote[n]), one
 * round-to-nearest fp32 operation; where vote[n] == 0 the bits of x[n] are left alone.
 *
 *  x     dev  [d] fp32, updated in place
 *  vote  dev, const [d] int8; any positive value counts as +1, any negative as -1
 */
S3GD_API s3gd_status s3gd_apply(float* x, const int8_t* vote, uint64_t d, float lr, void* stream);

/*
 * One whole step of Algorithm 1 after the local gradients exist (its "send",
 * "receive" and "x <-" lines): TopKSign per worker, majority vote, update of x.
 * Produces exactly what s3gd_topk_sign -> s3gd_majority_vote -> s3gd_apply
 * produce, without writing the intermediate message unless asked to.
 * With K == d this is signSGD with majority vote (Section 3.3, gamma = 1) and
 * runs as one streaming pass over the M sign planes.
 *
 *  x            dev  [d] fp32, updated in place
 *  grads        dev, const [M x d]
 *  opt_idx      dev or NULL  [M x K]            (as s3gd_topk_sign)
 *  opt_signbits dev or NULL  [M x ceil(K/32)]   (must be given together with opt_idx)
 *  opt_vote     dev or NULL  [d] int8
 */
S3GD_API s3gd_status s3gd_step(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr,
                      uint32_t* opt_idx, uint32_t* opt_signbits, int8_t* opt_vote,
                      void* ws, size_t ws_bytes, void* stream);

/*
 * The step with the two optional parts of Algorithm 1 around it:
 *
 *  - error compensation (Section 2.2, Eq. (5)-(6)), if opt_err != NULL: the selection works on
 *    g = grads + eta * err (fp32: the product rounded, then the sum rounded); afterwards err
 *    holds g with its K kept entries per worker set to +0, i.e. g - TopK(g);
 *  - momentum (Section 4.7), if opt_v != NULL: v <- mu * v + vote, x <- x - lr * v (every
 *    operation rounded once) instead of x <- x - lr * vote.  v and x change at every coordinate.
 *
 *  grads    dev, const [M x d]  this iteration's stochastic gradients (g~)
 *  opt_err  dev or NULL [M x d]  error memory e, updated in place (all zero before the first step)
 *  opt_v    dev or NULL [d]      momentum v, updated in place
 *  everything else as for s3gd_step.  With both NULL the call is s3gd_step.
 *  K == d with error memory leaves err all zero (everything is kept); K == 0 leaves err = g.
 */
S3GD_API s3gd_status s3gd_step_ex(float* x, const float* grads, float* opt_err, float eta, float* opt_v, float mu,
                                  int M, uint64_t d, uint64_t K, float lr,
                                  uint32_t* opt_idx, uint32_t* opt_signbits, int8_t* opt_vote,
                                  void* ws, size_t ws_bytes, void* stream);

/*
 * Momentum form of the update for the unfused route (Section 4.7): v[n] <- fl(fl(mu * v[n]) + sgn(vote[n])),
 * x[n] <- fl(x[n] - fl(lr * v[n])).  x, v dev [d] fp32 in place; vote dev, const [d] int8.
 */
S3GD_API s3gd_status s3gd_apply_momentum(float* x, float* v, const int8_t* vote, uint64_t d, float mu, float lr,
                                         void* stream);

/*
 * Random-K variant (Section 3.4: RandKSign = sgn(RandK(g)); Algorithm 2 is Algorithm 1 with
 * TopKSign replaced by it).  Worker m keeps K coordinates drawn uniformly without repetition,
 * independently of the other workers and of earlier iterations.  The paper names no
 * generator; this library's is deterministic in (seed, step, m):
 *   key_r = mix(base + (r+1) * 0x9E3779B9),  base = seed ^ (m * 0x9E3779B9) ^ (step * 0x85EBCA6B)   (mod 2^32)
 *   mix(v): v ^= v>>16; v *= 0x7FEB352D; v ^= v>>15; v *= 0x846CA68B; v ^= v>>16             (mod 2^32)
 *   pi = 4 Feistel rounds on 2h bits, h minimal with 2^(2h) >= d:  (L, R) <- (R, L ^ (mix(R ^ key_r) & (2^h - 1))),
 *        applied again while the value is >= d (cycle walking)
 * and the kept coordinates are pi(0), ..., pi(K-1) IN THAT ORDER (not ascending): entry j of
 * out_idx is pi(j) and sign bit j is the IEEE sign bit of that entry.  A receiver that knows
 * (seed, step, m) can regenerate the indices, so only the sign words need to travel.
 * s3gd_majority_vote accepts this message as it is.
 *
 *  s3gd_randk_sign   arguments as s3gd_topk_sign plus seed, step
 *  s3gd_step_randk   arguments as s3gd_step plus seed, step; equals
 *                    s3gd_randk_sign -> s3gd_majority_vote -> s3gd_apply
 * K == 0 writes nothing; K == d keeps everything (the step is then signSGD with majority vote).
 * No error compensation: Section 3.4 notes that random selection does not need it.
 */
S3GD_API s3gd_status s3gd_randk_sign(const float* grads, int M, uint64_t d, uint64_t K, uint32_t seed, uint32_t step,
                                     uint32_t* out_idx, uint32_t* out_signbits,
                                     void* ws, size_t ws_bytes, void* stream);
S3GD_API s3gd_status s3gd_step_randk(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr,
                                     uint32_t seed, uint32_t step,
                                     uint32_t* opt_idx, uint32_t* opt_signbits, int8_t* opt_vote,
                                     void* ws, size_t ws_bytes, void* stream);

/*
 * Waits for `stream`, then reports what the kernels of earlier calls on this
 * workspace recorded: S3GD_OK, S3GD_ERR_INDEX_RANGE or S3GD_ERR_INTERNAL.
 * The record is cleared by the next s3gd_topk_sign / s3gd_majority_vote / s3gd_step.
 * If info is not NULL (host, 8 x uint32) it receives diagnostic counters:
 *   [0] status word  [1] rows that took the exact multi-pass route
 *   [2] out-of-range indices skipped  [3] rows whose selection size != K
 *   [4] largest candidate count of a row  [5..7] reserved (0)
 */
S3GD_API s3gd_status s3gd_device_status(const void* ws, void* stream, uint32_t* info);
/* The same without the counters: s3gd_device_status(ws, stream, NULL). */
S3GD_API s3gd_status s3gd_last_device_status(const void* ws, void* stream);

/*
 * Test hooks for the exactness safety net (the paper has no counterpart).
 *
 * For 0 < K <= d/4 the selection reads each gradient row once: a threshold tau_lo taken at a
 * fixed rank of a 65,536-entry sample of the row filters the row, and the top K are then found
 * among the survivors.  A row whose filter kept fewer than K entries (threshold too high) or
 * more than the workspace has room for (too low) is redone exactly over the whole row; that
 * decision is taken per row on the device, and with a sound sampling rank it is almost never
 * needed.  The fused step without optional outputs, for K around 0.4 % of d and more, also takes
 * a second threshold tau_hi from the sample, at a rank BELOW the expected one: entries at or
 * above it are the largest of the row, so they vote during the filter pass itself, and only
 * the band between the two thresholds is listed.  If more than K entries turn out to lie at or
 * above tau_hi the row is redone too, and the votes that should not have been cast are taken back.
 * These two calls are s3gd_topk_sign and s3gd_step with the ranks given by the caller, so that
 * a test can force every one of these failures on ordinary data:
 *   sample_rank   rank of tau_lo; 1 puts it at the largest sampled magnitude (too few survivors),
 *                 a rank near 65,536 at the smallest (too many); 0 = the library's own rank
 *   prevote_rank  rank of tau_hi; a rank well above 65,536 * K / d makes more than K entries
 *                 vote early; 0 = the library's own rank
 * The results must be, and are tested to be, identical to those of the ordinary calls; info[1] of
 * s3gd_device_status counts the rows that were redone.  Workspace as for the ordinary calls.
 */
S3GD_API s3gd_status s3gd_debug_topk_sign(const float* grads, int M, uint64_t d, uint64_t K,
                                          uint32_t* out_idx, uint32_t* out_signbits,
                                          void* ws, size_t ws_bytes, void* stream, uint32_t sample_rank);
S3GD_API s3gd_status s3gd_debug_step(float* x, const float* grads, int M, uint64_t d, uint64_t K, float lr,
                                     uint32_t* opt_idx, uint32_t* opt_signbits, int8_t* opt_vote,
                                     void* ws, size_t ws_bytes, void* stream, uint32_t sample_rank,
                                     uint32_t prevote_rank);

/*
 * The step when the workers of Algorithm 1 sit on several GPUs.  The library does not communicate:
 * these are the pieces on either side of the caller's collective.
 *
 * s3gd_vote_apply -- majority vote (Section 2.2 "Majority vote") over a message gathered from several
 * senders, fused with the update (Eq. (7)); equals s3gd_majority_vote + s3gd_apply over all workers.
 *   msg           dev, const  n_groups pieces, group_stride uint32 words apart; a piece is what one sender
 *                             produced with s3gd_topk_sign / s3gd_randk_sign for its M_group workers:
 *                             indices [M_group x K] directly followed by sign words [M_group x ceil(K/32)]
 *                             (an all-gather of equal pieces has group_stride = M_group * (K + ceil(K/32)))
 *   ws            dev         >= s3gd_workspace_bytes(n_groups * M_group, d, K)
 *   opt_vote      dev or NULL [d] int8
 * Contract: no worker repeats an index (true of the two producers above); with up to 127 workers the
 * votes are then counted in bytes.  A message that may repeat indices goes to s3gd_majority_vote.
 * An index >= d is skipped and S3GD_ERR_INDEX_RANGE recorded, as there.
 *
 * s3gd_vote_counts -- the sums before the sign, for a server that is split over GPUs by coordinate
 * range: every GPU sums the votes of its own workers, the sums are added across GPUs (reduce-scatter),
 * each GPU takes the sign of its range.  count[n] = sum over the M workers of their vote on n.
 *   out_counts      dev  [d_padded] counts, d_padded >= d a multiple of 4 (coordinates beyond d hold zero)
 *   bytes_per_count 4: int32 sums.  1: one byte per coordinate holding 128 + sum (M <= 127, same contract
 *                   as above); adding R such buffers bytewise modulo 256 gives 128 * R + total, which
 *                   s3gd_encode_vote2 undoes when told R, provided the total stays within +-127.
 *   opt_bad_count   dev or NULL  receives the number of indices >= d that were skipped
 *
 * s3gd_encode_vote2 / s3gd_apply_vote2 -- the server's message in a dense form of two bits per
 * coordinate (bit 0: moved, bit 1: negative; 0 -> 00, +1 -> 01, -1 -> 11; sixteen coordinates per uint32
 * word, lowest bits first, padding 00), a sixteenth of the int32 sums and a quarter of the int8 vote.
 * The paper counts |N^t| + |N^t| log2(N / |N^t|) <= N bits for this message with an index code; two
 * bits each is the form a GPU can write and read at memory speed.
 *   src, src_kind   dev, const  n values: kind 0 int32 sums, kind 1 bytes as written by s3gd_vote_counts
 *                   and summed over n_summed buffers, kind 2 an int8 vote (any positive = +1, negative = -1)
 *   out_words       dev  [ceil(n / 16)]
 *   s3gd_apply_vote2: x[n] <- fl32(x[n] - lr * vote[n]) from the words, one rounding, unmoved bits left
 *                   alone; opt_vote (dev or NULL, [d] int8) receives the decoded vote.
 *
 * s3gd_encode_vote_sparse / s3gd_apply_vote_sparse -- the same message in the sparse form the paper's
 * count assumes (Section 2.2: only the union of the workers' supports is sent): the coordinates with a
 * non-zero vote, ascending, and one sign bit each, in the layout of a worker's message.
 *   src, src_kind, n_summed, n   as for s3gd_encode_vote2: the votes (or sums) of n consecutive coordinates
 *   index_base      the coordinate of src[0] (a server that owns one range of the coordinates passes its start)
 *   out_piece       dev  [1 + cap + ceil(cap / 32)] uint32: the number of non-zero votes, then up to cap
 *                   indices (index_base + position, ascending), then their sign words (bit j belongs to
 *                   index j, lowest bits first, 1 = negative, padding 0).  If there are more than cap
 *                   non-zero votes the count says so and only the first cap are listed: the caller compares.
 *   ws, ws_bytes    dev  scratch of s3gd_sparse_workspace_bytes(n) bytes, 4-byte aligned
 *   s3gd_apply_vote_sparse: applies n_pieces such pieces, piece_stride uint32 words apart (an all-gather of
 *                   equal pieces), to x; an index >= d is skipped and counted in opt_bad_count (dev or NULL).
 *                   A piece whose count exceeds cap is applied as far as it is listed.
 */
S3GD_API s3gd_status s3gd_vote_apply(float* x, const uint32_t* msg, int n_groups, uint64_t group_stride, int M_group,
                                     uint64_t K, uint64_t d, float lr, int8_t* opt_vote,
                                     void* ws, size_t ws_bytes, void* stream);
S3GD_API s3gd_status s3gd_vote_counts(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K, uint64_t d,
                                      uint64_t d_padded, void* out_counts, int bytes_per_count,
                                      uint32_t* opt_bad_count, void* stream);
S3GD_API s3gd_status s3gd_encode_vote2(const void* src, int src_kind, uint32_t n_summed, uint64_t n,
                                       uint32_t* out_words, void* stream);
S3GD_API s3gd_status s3gd_apply_vote2(float* x, const uint32_t* words, uint64_t d, float lr, int8_t* opt_vote,
                                      void* stream);
S3GD_API size_t s3gd_sparse_workspace_bytes(uint64_t n);
S3GD_API s3gd_status s3gd_encode_vote_sparse(const void* src, int src_kind, uint32_t n_summed, uint64_t n,
                                             uint32_t index_base, uint32_t cap, uint32_t* out_piece,
                                             void* ws, size_t ws_bytes, void* stream);
S3GD_API s3gd_status s3gd_apply_vote_sparse(float* x, const uint32_t* pieces, int n_pieces, uint64_t piece_stride,
                                            uint32_t cap, uint64_t d, float lr, uint32_t* opt_bad_count,
                                            void* stream);

/*
 * Majority vote without any caller-provided scratch (the paper has no counterpart: this is
 * a convenience of this library, same result as s3gd_majority_vote).
 *
 * For callers that cannot allocate device memory where they vote -- code running inside
 * another framework's callback that must not call into its allocator, a plug-in that is
 * handed nothing but input and output buffers, a process whose device memory is already
 * fully owned by a pool it does not control.  The d int32 counters live in a fixed array
 * inside this library's GPU code (16 MiB + 256 bytes per GPU), so d is limited:
 * s3gd_noalloc_max_d() = 4,194,304 coordinates; a larger d returns S3GD_ERR_TOO_LARGE and
 * nothing is enqueued.  The call itself calls no allocation routine and frees nothing.
 *
 * When the array's memory is taken: not when the library is loaded into the process.  The
 * CUDA runtime loads GPU code lazily by default, so the 16 MiB (and the code of the two
 * kernels the call uses) are reserved on a device by the FIRST call made there, and are then
 * held until the process exits.  Make that first call -- any small vote will do -- while the
 * device still has that much free memory; if it does not, the first call returns
 * S3GD_ERR_CUDA and can be repeated later.  Running the process with
 * CUDA_MODULE_LOADING=EAGER moves the reservation to the creation of the CUDA context.
 *
 *  idx, signbits, M, K, d, out_vote   as for s3gd_majority_vote (dev pointers)
 *  opt_bad_count  dev or NULL  receives the number of indices >= d that were skipped
 *
 * The first call on each device also looks up the device address of the built-in array (a
 * runtime query) with that device current; make that first call outside any stream
 * capture.  All calls on a device share the one array: it is cleared at the start of every
 * call, so results never depend on earlier calls, but two calls that may run on the GPU at
 * the same time (different streams) race on it -- serialise them.  Not thread-safe: do not
 * make the first call on a device from two host threads at once.
 */
S3GD_API uint64_t s3gd_noalloc_max_d(void);
S3GD_API s3gd_status s3gd_majority_vote_noalloc(const uint32_t* idx, const uint32_t* signbits, int M, uint64_t K,
                                                uint64_t d, int8_t* out_vote, uint32_t* opt_bad_count,
                                                void* stream);

/*
 * Measurement aid (the paper reports no timings; this has no counterpart there).
 * Between s3gd_profile_begin(max_steps) and s3gd_profile_end(), every s3gd_step call of
 * this process records CUDA events on its stream at its phase boundaries, for at most
 * max_steps calls.  s3gd_profile_end synchronises the device and writes, for each recorded
 * call, 5 durations in milliseconds to out_ms (host, [max_steps x 5], may be NULL):
 *   [0] clear counters + sampled threshold   [1] filter pass over the gradients
 *   [2] radix passes for the exact threshold [3] per-tile counts, scan, ordered emission
 *   [4] sign of the counters + update of x   (K == d: [4] is the whole sign-plane pass)
 * *n_steps (host) receives the number of recorded calls and *launches (host) the number
 * of kernels this library enqueued since s3gd_profile_begin.  Not thread-safe; one
 * profiling session at a time.  The events are created and destroyed by these two calls.
 */
S3GD_API s3gd_status s3gd_profile_begin(int max_steps);
/* The same, but only the two events around the filter pass are recorded ([1] is valid, the other
 * durations are reported as 0): event records between kernels cost a few microseconds each, so this
 * is the form to leave on while a step is being timed as a whole. */
S3GD_API s3gd_status s3gd_profile_begin_filter(int max_steps);
/* The same with only every `every`-th step call recorded (the first one is), at most max_steps of them: a
 * sample of the filter pass's duration over a long run at 1 / every of the events' cost.  every >= 1. */
S3GD_API s3gd_status s3gd_profile_begin_filter_every(int max_steps, int every);
S3GD_API s3gd_status s3gd_profile_end(float* out_ms, int* n_steps, uint64_t* launches);

#ifdef __cplusplus
}
#endif
#endif /* S3GD_H_ */

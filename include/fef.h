/*
 * fef.h - C ABI of the B200 (sm_100a) speculative-verification library for
 * FeF-DLLM decoding.
 *
 * The library implements, on one GPU, the verification loop of the paper's
 * full-sequence decoding algorithm (Algorithm 2, the loop over a window's
 * positions; Section 3.2 on speculative decoding; the residual law defined before
 * Algorithm 2) for B independent speculative windows at once, and the
 * low-confidence selection LowConf_{n_rm} of the same algorithm.
 *
 * Conventions
 *  - Pointers marked "device" must be device memory of the current CUDA device;
 *    the caller owns every buffer.  The library allocates nothing, keeps no
 *    state between calls and never synchronises: all work (three kernels per
 *    verification call, the first of which clears the counters it needs and the
 *    status word) is enqueued on `cuda_stream` (a cudaStream_t passed as void*;
 *    NULL = the default stream).
 *  - The return value reports what the host can see (bad arguments, launch
 *    failures).  Errors that only the data reveals are written to
 *    `*device_status` by the kernels; nothing ever traps.
 *  - No CPU fallback exists: without a CUDA device every compute entry point
 *    returns FEF_ERR_CUDA.
 */
#ifndef FEF_H
#define FEF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FEF_OK = 0,
    FEF_ERR_INVALID_ARG = 1, /* null pointer, size out of range, temperature < 0 or NaN   */
    FEF_ERR_DTYPE = 2,       /* dtype is neither FEF_F32 nor FEF_BF16                     */
    FEF_ERR_ALIGNMENT = 3,   /* logit base pointers or row pitch not 16-byte multiples    */
    FEF_ERR_WORKSPACE = 4,   /* workspace missing, misaligned (256 B) or too small        */
    FEF_ERR_CUDA = 5,        /* CUDA runtime error (see cudaGetLastError), or no device   */
    FEF_ERR_TIMEOUT = 6,     /* device: a bounded wait inside a kernel ran out            */
    FEF_ERR_NONFINITE = 7,   /* device: NaN or +inf logit, or a row that is all -inf      */
    FEF_ERR_TOKEN_RANGE = 8, /* device: a draft token outside [0, V)                      */
    FEF_ERR_TOO_LARGE = 9    /* fef_spec_verify_static: sizes exceed its built-in scratch  */
} fef_status;

typedef enum { FEF_F32 = 0, FEF_BF16 = 1 } fef_dtype;

/* Largest window and selection sizes accepted. */
#define FEF_MAX_B 65535
#define FEF_MAX_K 64
#define FEF_MAX_REMASK_L 8192
/* Token id of a masked (unresolved) position in the decode-loop state. */
#define FEF_MASK_TOKEN (-1)

/* Human-readable name of a status value (static storage, never NULL). */
const char* fef_status_string(fef_status s);

/*
 * Bytes of device scratch fef_spec_verify needs for these sizes on the current
 * CUDA device (it depends on the device's SM count).  Returns 0 for invalid
 * sizes or when no device is available.  The scratch must be 256-byte aligned;
 * its contents need not be initialised (the call clears the counters it keeps
 * there) and are meaningless afterwards.  Two calls that may overlap on the GPU
 * need separate scratch buffers.
 */
size_t fef_spec_verify_workspace_bytes(int B, int K, int V, fef_dtype dt);

/*
 * One verification call over B speculative windows of K positions
 * (Algorithm 2, the loop over the window's positions m up to the first rejection;
 * acceptance rule and correction of Section 3.2; residual law
 * pi' = [pi - rho]_+ / (1 - sum min{pi, rho})).
 *
 * With pi_i = softmax(target_logits[b,i,:] / T) and rho_i = softmax(draft_logits[b,i,:] / T),
 * for each window b, scanning i = 0, 1, ... < n_b (n_b = row_len[b], or K):
 *   u_i ~ U(0,1);  the draft x_i = draft_tokens[b,i] is accepted iff
 *   u_i <= min{1, pi_i(x_i) / rho_i(x_i)};  accepted: tokens[b,i] = x_i, conf[b,i] = pi_i(x_i).
 *   At the first rejection a: Z ~ pi'_a, tokens[b,a] = Z, conf[b,a] = pi_a(Z), stop.
 * accept_len[b] = a (or n_b when nothing was rejected).  Entries after the last
 * committed position get tokens = -1 and conf = -1.
 *
 * Temperature 0 is greedy: a draft is accepted iff it equals arg-max of the
 * target logits (lowest index on ties), the replacement is that arg-max, no
 * random numbers are used, draft_logits is not read, and conf is the T = 1
 * softmax probability of the committed token.
 *
 * Random numbers: Philox4x32-10 keyed by (seed low word, seed high word) with
 * counter ((stream << 30) | j, b, i, step).  Acceptance: stream 0, j = 0,
 * output word 0.  Residual draw: Gumbel-max over x with [pi - rho]_+ > 0 of
 * ln r_x - ln(-ln u_x), u_x from stream 1, j = x >> 2, output word x & 3;
 * lowest x on exact ties.  A word r maps to u = ((r >> 9) + 0.5) * 2^-23.
 * `step` must differ between calls that share a seed, or they reuse draws.
 *
 * Arguments
 *   draft_logits, target_logits  device, [B, K, ld] row-major, dtype `dt`; only the first
 *                    V entries of a row are read.  Base addresses and ld * sizeof(element)
 *                    must be multiples of 16 bytes.  -inf entries are legal (probability 0).
 *   draft_tokens     device, [B, K] int32, each in [0, V) for i < n_b
 *   row_len          device, [B] int32 in [0, K] (drafts actually present), or NULL = K everywhere
 *   B, K, V, ld      1 <= B <= FEF_MAX_B, 1 <= K <= FEF_MAX_K, V >= 1 (a row of at most 2^30 bytes),
 *                    ld >= V (elements)
 *   temperature      > 0 sampling, == 0 greedy; negative or NaN is FEF_ERR_INVALID_ARG
 *   accept_len       device out, [B] int32
 *   tokens           device out, [B, K] int32
 *   conf             device out, [B, K] float32
 *   workspace        device scratch of at least fef_spec_verify_workspace_bytes(...) bytes
 *   device_status    device out, [1] int32, or NULL.  Set to FEF_OK at the start of the call,
 *                    then to the largest device-side error.  Windows with a data error get
 *                    accept_len = -1 and no committed tokens; other windows are unaffected.
 *                    FEF_ERR_TIMEOUT (a bounded wait inside the streaming kernel ran out, which only
 *                    a fault elsewhere on the device can cause): no window is decided, every
 *                    accept_len is -1.
 *   cuda_stream      stream to enqueue on
 *
 * Calls that stream little (few rows) use kernels built for latency, larger ones a streaming kernel
 * built for bandwidth; the results are the same up to the rounding order of the row sums.
 */
fef_status fef_spec_verify(const void* draft_logits, const void* target_logits,
                           const int32_t* draft_tokens, const int32_t* row_len,
                           int B, int K, int V, int64_t ld, fef_dtype dt,
                           float temperature, uint64_t seed, uint32_t step,
                           int32_t* accept_len, int32_t* tokens, float* conf,
                           void* workspace, size_t workspace_bytes,
                           int32_t* device_status, void* cuda_stream);

/*
 * fef_spec_verify for drafts that come with their law's normaliser (same operation, same
 * citations: Algorithm 2's verification loop, Section 3.2).  `draft_log2_norm` is the
 * log2_norm output of fef_draft_sample for the same draft_logits and temperature:
 * rho_i(x) = 2^(l_x * log2(e) / T - draft_log2_norm[b,i]).  With it the draft rows need not be
 * read in full: only draft_logits[b,i,x_i] is, and the rejected position's row for the residual
 * draw, so a call moves half the bytes.  Results equal fef_spec_verify's up to the rounding of the
 * normaliser (confidences within 1e-5 relative, the same draws apart from near-ties).
 *   draft_log2_norm  device, [B, K] float64 (entries of positions i >= n_b are not read);
 *                    a NaN or infinite entry is FEF_ERR_NONFINITE for its window
 * Everything else as in fef_spec_verify; at temperature 0 the normalisers are not used.
 */
fef_status fef_spec_verify_with_draft_norm(const void* draft_logits, const void* target_logits,
                                           const int32_t* draft_tokens, const double* draft_log2_norm,
                                           const int32_t* row_len,
                                           int B, int K, int V, int64_t ld, fef_dtype dt,
                                           float temperature, uint64_t seed, uint32_t step,
                                           int32_t* accept_len, int32_t* tokens, float* conf,
                                           void* workspace, size_t workspace_bytes,
                                           int32_t* device_status, void* cuda_stream);

/*
 * fef_spec_verify with timing marks: the same operation (Algorithm 2's verification
 * loop) and the same results, and additionally up to four caller-created CUDA events
 * (cudaEvent_t passed as void*; NULL entries are skipped) are recorded on `cuda_stream`:
 * [0] before the streaming kernel, [1] after it, [2] and [3] after the kernel that follows
 * it (acceptance tests and residual draw are one launch; at temperature 0 the arg-max
 * scan).  `stage_events` may be NULL.  Used to time the kernels separately; an event
 * between two kernels keeps the later one from starting early, so the whole call is a
 * little slower than fef_spec_verify.
 */
fef_status fef_spec_verify_profiled(const void* draft_logits, const void* target_logits,
                                    const int32_t* draft_tokens, const int32_t* row_len,
                                    int B, int K, int V, int64_t ld, fef_dtype dt,
                                    float temperature, uint64_t seed, uint32_t step,
                                    int32_t* accept_len, int32_t* tokens, float* conf,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* device_status, void* cuda_stream,
                                    void* const* stage_events);

/*
 * Host-buffer form of fef_spec_verify (same operation, same citations): every
 * array argument is HOST memory (pinned memory makes the copies asynchronous and
 * fast).  The call copies the inputs into `device_arena`, runs the verification
 * there, copies accept_len / tokens / conf and the device status word back, and
 * returns after synchronising `cuda_stream`.  At temperature 0 the draft logits
 * are not copied.
 *   device_arena        device scratch, 256-byte aligned, at least
 *                       fef_spec_verify_host_arena_bytes(B, K, V, ld, dt) bytes
 *   status_out          host out, may be NULL: the device status word of the call
 * The arena size is 0 for invalid sizes or when no CUDA device is available.
 */
size_t fef_spec_verify_host_arena_bytes(int B, int K, int V, int64_t ld, fef_dtype dt);
fef_status fef_spec_verify_host(const void* draft_logits, const void* target_logits,
                                const int32_t* draft_tokens, const int32_t* row_len,
                                int B, int K, int V, int64_t ld, fef_dtype dt,
                                float temperature, uint64_t seed, uint32_t step,
                                int32_t* accept_len, int32_t* tokens, float* conf,
                                int32_t* status_out,
                                void* device_arena, size_t device_arena_bytes, void* cuda_stream);

/*
 * fef_spec_verify for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, same results.)
 *
 * Some hosts of this library may not call cudaMalloc at the point where they verify:
 * code running inside someone else's memory plan (an inference server that hands out
 * all device memory up front and forbids later allocations), plug-ins that receive
 * only input and output buffers, and code on a latency path where an allocation -
 * which may synchronise the device - is not acceptable.  For them the scratch that
 * fef_spec_verify takes as `workspace` lives inside the library instead: a fixed
 * device array of FEF_STATIC_SCRATCH_BYTES that every GPU using the library holds from
 * the moment the library is loaded there until the process exits.  The call itself
 * allocates and frees nothing.
 *
 * Arguments are those of fef_spec_verify without workspace / workspace_bytes; the
 * caller still owns all inputs and outputs.
 *   - Sizes whose scratch need (fef_spec_verify_workspace_bytes) exceeds
 *     FEF_STATIC_SCRATCH_BYTES are refused with FEF_ERR_TOO_LARGE and nothing is
 *     launched.  The shape B = 64, K = 32, V = 126464 needs about 0.2 MB.
 *   - The first call on each device looks up the array's device address (one runtime
 *     query).  If nothing of this library has run on that device before, that is also
 *     the moment the CUDA runtime loads the library's device code there and reserves the
 *     array with it, so make one warm-up call per device at start-up, outside any stream
 *     capture; later calls neither allocate nor query.
 *   - All calls on a device share the one array.  It keeps whatever the previous call
 *     left; no call depends on that content.  Two calls whose kernels can overlap on
 *     the GPU (different streams, no ordering between them) race on it and give
 *     undefined results: keep calls of this entry point ordered, or use fef_spec_verify
 *     with separate workspaces.
 */
#define FEF_STATIC_SCRATCH_BYTES (8u << 20)
fef_status fef_spec_verify_static(const void* draft_logits, const void* target_logits,
                                  const int32_t* draft_tokens, const int32_t* row_len,
                                  int B, int K, int V, int64_t ld, fef_dtype dt,
                                  float temperature, uint64_t seed, uint32_t step,
                                  int32_t* accept_len, int32_t* tokens, float* conf,
                                  int32_t* device_status, void* cuda_stream);

/*
 * Draft-token sampling (Algorithm 2, the step that draws the window's draft tokens from the
 * draft laws; Section 3.2): for every window b and position i < n_b one draw
 *   draft_tokens[b,i] ~ rho_i = softmax(draft_logits[b,i,:] / T),
 * taken by Gumbel-max: arg-max over x of l_x / T - ln(-ln u_x) among the entries with
 * l_x > -inf, lowest x on exact ties.  u_x comes from Philox4x32-10 keyed like fef_spec_verify,
 * stream 2: counter ((2 << 30) | (x >> 2), b, i, step), output word x & 3,
 * u = ((r >> 9) + 0.5) * 2^-23.  Temperature 0: arg-max of the logits (lowest index on ties),
 * no random numbers.  Pass the same `seed` and `step` as to the fef_spec_verify call that
 * checks these drafts: the two calls use different Philox streams.
 *
 * Arguments
 *   draft_logits   device, [B, K, ld] row-major, dtype `dt`, same layout and alignment rules as
 *                  fef_spec_verify; -inf entries are legal (never drawn)
 *   row_len        device, [B] int32 in [0, K], or NULL = K everywhere
 *   draft_tokens   device out, [B, K] int32; -1 for i >= n_b and for positions with a data error
 *   log2_norm      device out, [B, K] float64, or NULL: log2 of sum_x 2^(l_x * log2(e) / T), the
 *                  normaliser of rho_i (rho_i(x) = 2^(l_x log2(e) / T - log2_norm)); at T = 0 the
 *                  T = 1 value; 0 where no token was drawn
 *   workspace      device scratch of at least fef_draft_sample_workspace_bytes(...) bytes,
 *                  256-byte aligned, contents need not be initialised
 *   device_status  device out, [1] int32, or NULL: FEF_OK, or FEF_ERR_NONFINITE when a used row
 *                  holds NaN or +inf or no finite logit (that position gets token -1)
 * Asynchronous on `cuda_stream`; one kernel.
 */
size_t fef_draft_sample_workspace_bytes(int B, int K, int V, fef_dtype dt);
fef_status fef_draft_sample(const void* draft_logits, const int32_t* row_len,
                            int B, int K, int V, int64_t ld, fef_dtype dt,
                            float temperature, uint64_t seed, uint32_t step,
                            int32_t* draft_tokens, double* log2_norm,
                            void* workspace, size_t workspace_bytes,
                            int32_t* device_status, void* cuda_stream);

/*
 * Draft draws and the target laws' normalisers in one pass (Algorithm 2: the draft tokens are drawn
 * from rho, then the target laws pi are needed at them): fef_draft_sample that reads the target
 * logits of the same rows alongside and also returns
 *   target_log2_norm  device out, [B, K] float64: log2 of sum_x 2^(l^p_x * log2(e) / T) per position
 *                     (NaN where the target row holds NaN or +inf or no finite logit; 0 for i >= n_b),
 * so that both tensors are read once, by one kernel.  fef_spec_verify_with_norms then verifies
 * without streaming anything: it takes both normalisers, reads the two logits at each draft token and
 * the rejected position's rows for the residual draw.  Results equal fef_spec_verify's up to the
 * rounding of the normalisers (confidences within 1e-5 relative, the same draws apart from
 * near-ties).  device_round: NULL, or the device-resident round counter of the *_at_round calls.
 * At temperature 0 fef_spec_verify_with_norms ignores the normalisers and runs as fef_spec_verify does.
 * Workspaces: fef_draft_sample_workspace_bytes / fef_spec_verify_workspace_bytes.
 */
fef_status fef_draft_sample_with_target(const void* draft_logits, const void* target_logits, const int32_t* row_len,
                                        int B, int K, int V, int64_t ld, fef_dtype dt,
                                        float temperature, uint64_t seed, uint32_t step, const uint32_t* device_round,
                                        int32_t* draft_tokens, double* draft_log2_norm, double* target_log2_norm,
                                        void* workspace, size_t workspace_bytes,
                                        int32_t* device_status, void* cuda_stream);
fef_status fef_spec_verify_with_norms(const void* draft_logits, const void* target_logits, const int32_t* draft_tokens,
                                      const double* draft_log2_norm, const double* target_log2_norm,
                                      const int32_t* row_len,
                                      int B, int K, int V, int64_t ld, fef_dtype dt,
                                      float temperature, uint64_t seed, uint32_t step, const uint32_t* device_round,
                                      int32_t* accept_len, int32_t* tokens, float* conf,
                                      void* workspace, size_t workspace_bytes,
                                      int32_t* device_status, void* cuda_stream);

/*
 * LowConf_k of Algorithm 2 (the selection of the n_rm least confident positions of C^(s)
 * at the end of a denoising step): for every batch row the k candidate positions of lowest
 * confidence.
 *
 *   conf       device, [B, L] float32 confidences
 *   mask       device, [B, L] uint8; a position is a candidate iff mask != 0
 *   B, L, k    B >= 1, 1 <= L <= FEF_MAX_REMASK_L, k >= 0
 *   positions  device out, [B, k] int32: candidates ordered by (conf ascending, index
 *              ascending), padded with -1 when fewer than k candidates exist
 *   count      device out, [B] int32 = min(k, number of candidates)
 * -0 and +0 compare equal; NaN sorts after every number.
 */
fef_status fef_remask_select(const float* conf, const uint8_t* mask, int B, int L, int k,
                             int32_t* positions, int32_t* count, void* cuda_stream);

/*
 * Host-buffer form of fef_remask_select (same operation): conf, mask, positions
 * and count are HOST memory; the call stages them through `device_arena`
 * (256-byte aligned, at least fef_remask_select_host_arena_bytes(B, L, k) bytes)
 * and returns after synchronising `cuda_stream`.
 */
size_t fef_remask_select_host_arena_bytes(int B, int L, int k);
fef_status fef_remask_select_host(const float* conf, const uint8_t* mask, int B, int L, int k,
                                  int32_t* positions, int32_t* count,
                                  void* device_arena, size_t device_arena_bytes, void* cuda_stream);

/*
 * Bookkeeping of the full-sequence decoding loop (Algorithm 2) on the device.  State of B
 * sequences of L positions: tokens [B, L] int32 (FEF_MASK_TOKEN = unresolved), conf [B, L]
 * float32 (-1 where unresolved), in_step [B, L] uint8 (1 = committed during the current
 * denoising step, the set C^(s)).  All pointers are device memory; every call is one small
 * kernel on `cuda_stream`.  1 <= L <= 2^24, 1 <= K <= FEF_MAX_K.
 *
 * fef_loop_next_window  (Algorithm 2: the ordered set J_t of unresolved positions and the window
 *   size b = min{k, L_t}): window_pos [B, K] = the first K unresolved positions of each row in
 *   increasing order, -1 padded; row_len [B] = min(K, L_t); unresolved [B] = L_t.
 * fef_loop_verification_inputs  (Algorithm 2: the verification inputs X^(j_m), i.e. the verified
 *   prefix plus the drafts of the window's earlier positions): inputs [B, K, L]; row m is the
 *   sequence with the drafts of the window's positions 0 .. min(m, row_len) - 1 written in.
 * fef_loop_commit  (Algorithm 2: the write-back of an accepted draft or of the corrected token
 *   with its confidence into X and C^(s); later drafts of the window are dropped): writes the
 *   first min(accept_len + 1, row_len) entries of out_tokens / out_conf (outputs of
 *   fef_spec_verify) to their positions, marks them in in_step; committed [B] = that count, or -1
 *   (nothing written) for a window with accept_len = -1.
 * fef_loop_remask  (Algorithm 2: re-corruption of the positions LowConf selected, with the
 *   absorbing-state forward kernel): the first min(count[b], k) entries of positions [B, k]
 *   (output of fef_remask_select) go back to FEF_MASK_TOKEN with conf -1; in_step is cleared for
 *   the next denoising step.
 */
fef_status fef_loop_next_window(const int32_t* tokens, int B, int L, int K,
                                int32_t* window_pos, int32_t* row_len, int32_t* unresolved, void* cuda_stream);
fef_status fef_loop_verification_inputs(const int32_t* tokens, const int32_t* window_pos, const int32_t* row_len,
                                        const int32_t* draft_tokens, int B, int L, int K,
                                        int32_t* inputs, void* cuda_stream);
fef_status fef_loop_commit(const int32_t* window_pos, const int32_t* row_len, const int32_t* accept_len,
                           const int32_t* out_tokens, const float* out_conf, int B, int L, int K,
                           int32_t* tokens, float* conf, uint8_t* in_step, int32_t* committed, void* cuda_stream);
fef_status fef_loop_remask(const int32_t* positions, const int32_t* count, int B, int L, int k,
                           int32_t* tokens, float* conf, uint8_t* in_step, void* cuda_stream);

/*
 * The same calls with the step number completed on the device, for loops that are replayed as a
 * CUDA graph (the inner loop of Algorithm 2 over the unresolved positions without a host round trip: a
 * captured round keeps its by-value arguments, so the number that makes every round's random
 * numbers distinct has to live in device memory).  The step used is step + *device_round, read
 * when the kernels run.  device_round: device, [1] uint32, required (NULL is
 * FEF_ERR_INVALID_ARG); it must not change between the draft draws of a round and their
 * verification.  fef_loop_advance_round adds one to it on `cuda_stream`; when `unresolved`
 * (device, [B] int32, the output of fef_loop_next_window; may be NULL) is given it does so only
 * if some row still had an unresolved position, so that replayed rounds with nothing left to
 * do take no number.
 * fef_spec_verify_at_round takes draft_log2_norm as fef_spec_verify_with_draft_norm does, or NULL
 * to stream the draft rows as fef_spec_verify does.  Everything else as in the plain calls.
 */
fef_status fef_draft_sample_at_round(const void* draft_logits, const int32_t* row_len,
                                     int B, int K, int V, int64_t ld, fef_dtype dt,
                                     float temperature, uint64_t seed, uint32_t step, const uint32_t* device_round,
                                     int32_t* draft_tokens, double* log2_norm,
                                     void* workspace, size_t workspace_bytes,
                                     int32_t* device_status, void* cuda_stream);
fef_status fef_spec_verify_at_round(const void* draft_logits, const void* target_logits,
                                    const int32_t* draft_tokens, const double* draft_log2_norm,
                                    const int32_t* row_len,
                                    int B, int K, int V, int64_t ld, fef_dtype dt,
                                    float temperature, uint64_t seed, uint32_t step, const uint32_t* device_round,
                                    int32_t* accept_len, int32_t* tokens, float* conf,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* device_status, void* cuda_stream);
fef_status fef_loop_advance_round(uint32_t* device_round, const int32_t* unresolved, int B, void* cuda_stream);

/*
 * Vocabulary-parallel verification: fef_spec_verify (Algorithm 2's verification loop, the laws of
 * Section 3.2, the residual law defined before Algorithm 2) when each of `ranks` GPUs holds a
 * slice [vocab_offset, vocab_offset + V_local) of every logit row, as logits leave a
 * tensor-parallel output layer.  Sampling mode only (temperature > 0).  The library does the
 * per-rank work; the caller moves the two small messages between ranks (an all-gather each):
 *
 *   1. fef_vp_local_stats     streams this rank's slices once and writes, per position, six
 *                             doubles: reference and sum of both laws over the slice, and the two
 *                             logits at the draft token on the rank that holds it (NaN elsewhere).
 *                             stats: device out, [B*K][6] float64.
 *      -> all-gather to stats_all [ranks][B*K][6]
 *   2. fef_vp_accept          folds the ranks' numbers into pi_i(x_i), rho_i(x_i), applies the
 *                             acceptance tests (same random numbers as fef_spec_verify) and writes
 *                             accept_len, the accepted tokens and confidences, and per window the
 *                             rejected position with its normalisers (`tasks`, device, opaque,
 *                             fef_vp_task_bytes(B) bytes).  Every rank computes the same.
 *   3. fef_vp_local_residual  Gumbel-max over this rank's slice of every rejected row with the
 *                             global ids' random numbers; writes its best candidate per window.
 *                             candidates: device out, [B] records of 16 bytes (float64 score,
 *                             float32 target logit, int32 global id); windows without a rejection
 *                             are left untouched.
 *      -> all-gather to candidates_all [ranks][B]
 *   4. fef_vp_finish          largest score wins (lowest id on ties; if [pi - rho]_+ is zero
 *                             everywhere, the largest target logit): writes tokens[b, a_b] and
 *                             conf[b, a_b].
 *
 * Results equal fef_spec_verify's on the concatenated rows up to the rounding order of the sums.
 * vocab_offset must be a multiple of 8; slices must tile [0, V_total) without overlap; workspace:
 * fef_spec_verify_workspace_bytes(B, K, V_local, dt) bytes per rank, shared by steps 1 and 3.
 * Arguments not listed are as in fef_spec_verify; step 1 needs neither seed nor step.
 */
size_t fef_vp_task_bytes(int B);
fef_status fef_vp_local_stats(const void* draft_slice, const void* target_slice,
                              const int32_t* draft_tokens, const int32_t* row_len,
                              int B, int K, int V_local, int64_t ld, fef_dtype dt,
                              float temperature, int vocab_offset, double* stats,
                              void* workspace, size_t workspace_bytes,
                              int32_t* device_status, void* cuda_stream);
fef_status fef_vp_accept(const double* stats_all, int ranks,
                         const int32_t* draft_tokens, const int32_t* row_len,
                         int B, int K, int V_total, fef_dtype dt,
                         float temperature, uint64_t seed, uint32_t step,
                         int32_t* accept_len, int32_t* tokens, float* conf, void* tasks,
                         int32_t* device_status, void* cuda_stream);
fef_status fef_vp_local_residual(const void* draft_slice, const void* target_slice, void* tasks,
                                 int B, int K, int V_local, int64_t ld, fef_dtype dt,
                                 float temperature, uint64_t seed, uint32_t step, int vocab_offset,
                                 void* candidates, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream);
fef_status fef_vp_finish(const void* candidates_all, int ranks, const void* tasks,
                         int B, int K, fef_dtype dt, float temperature,
                         int32_t* tokens, float* conf, void* cuda_stream);

/*
 * Verification straight from hidden states (Section 3.2: the draft law rho^i and the target law pi^i
 * are outputs of the model, i.e. softmax of hidden state x output-layer weight; Algorithm 2's loop
 * over the window's positions and the residual law defined before it, as in fef_spec_verify).
 *
 *   logits^p[b,i,v] = sum_k target_hidden[b*K+i, k] * weight[v, k]      (and ^q with draft_hidden),
 * accumulated in binary32 on the tensor cores from the bfloat16 inputs and never rounded to
 * bfloat16 or written out: the product's epilogue keeps, per row and vocabulary chunk, the softmax
 * partial sums and the logit at the draft token.  From there the call is fef_spec_verify on those
 * binary32 logits: same acceptance rule, same random numbers (Philox counters as documented there),
 * same outputs and sentinels.  The residual draw recomputes the logits of the rejected positions
 * (2 B rows) with a second, small product.  Sampling mode only (temperature > 0).
 *
 *   draft_hidden, target_hidden  device, [B*K, d] bfloat16 row-major, 16-byte aligned
 *   weight                       device, [V, d] bfloat16 row-major (the output layer), 16-byte aligned
 *   d                            hidden width, a multiple of 8
 *   workspace                    device scratch of fef_lmhead_verify_workspace_bytes(B, K, V, d) bytes
 *                                (it holds, among others, the 2 B rows of binary32 logits), 256-byte aligned
 * Everything else as in fef_spec_verify.  Asynchronous on `cuda_stream`; five kernels.
 *
 * fef_lmhead_logits writes the same binary32 logits for arbitrary rows, logits[r, v] for r < rows
 * (ldo >= V elements per row, a multiple of 4): what the verification above sees, for inspection.
 */
size_t fef_lmhead_verify_workspace_bytes(int B, int K, int V, int d);
fef_status fef_lmhead_verify(const void* draft_hidden, const void* target_hidden, const void* weight,
                             const int32_t* draft_tokens, const int32_t* row_len,
                             int B, int K, int V, int d,
                             float temperature, uint64_t seed, uint32_t step,
                             int32_t* accept_len, int32_t* tokens, float* conf,
                             void* workspace, size_t workspace_bytes,
                             int32_t* device_status, void* cuda_stream);
fef_status fef_lmhead_logits(const void* hidden, const void* weight, int rows, int V, int d,
                             float* logits, int64_t ldo, int32_t* device_status, void* cuda_stream);

/*
 * Seeded synthetic logits made on the device (benchmarks and tests of the decoding loop; they stand
 * in for the two model calls of Algorithm 2 and hold none of the method's arithmetic):
 *   draft  = draft_std * N(0,1), plus `boost` with probability boost_fraction (in steps of 1/512),
 *   target = draft + noise_std * N(0,1),
 * every element a pure function of (seed, round + *device_round, row, vocabulary id) through
 * Philox4x32-10 and Box-Muller, rounded to the storage type.  [B, K, ld] row-major as in
 * fef_spec_verify; ld must cover whole 16-byte vectors (ld >= V rounded up to 8 bfloat16 / 4 float32
 * elements): the entries between V and that bound are written too.  device_round may be NULL.
 */
fef_status fef_synth_logits(void* draft_logits, void* target_logits, int B, int K, int V, int64_t ld, fef_dtype dt,
                            float draft_std, float noise_std, float boost_fraction, float boost,
                            uint64_t seed, uint32_t round, const uint32_t* device_round, void* cuda_stream);

/*
 * The whole decoding loop of Algorithm 2 as ONE submission, with fef_synth_logits in the place of
 * the two model calls: n_steps denoising steps over B sequences of L positions; every round is
 * window -> (at the end of a step: LowConf_k and re-masking) -> logits -> draft draws with the target
 * normalisers -> verification -> commit, until nothing is unresolved after the last step.  The
 * rounds are the body of a CUDA graph WHILE node whose condition a kernel of the round sets, so the
 * host neither reads anything back nor submits anything between rounds.
 *   tokens, conf, in_step  device, [B, L]: the state; pass all positions masked (FEF_MASK_TOKEN, -1, 0)
 *                          to decode from scratch
 *   device_round           device, [1] uint32: the round counter (random numbers of round r use step r);
 *                          start it at 0; on return it holds the number of rounds run
 *   L <= FEF_MAX_REMASK_L; temperature > 0; remask_k >= 0
 *   workspace              fef_loop_run_synthetic_workspace_bytes(...) bytes (it holds the two logit
 *                          tensors of a round), 256-byte aligned
 * The call builds, launches and destroys the graph and returns after synchronising `cuda_stream`.
 */
size_t fef_loop_run_synthetic_workspace_bytes(int B, int L, int K, int V, fef_dtype dt, int remask_k);
fef_status fef_loop_run_synthetic(int B, int L, int K, int V, fef_dtype dt, float temperature, uint64_t seed,
                                  int n_steps, int remask_k, float draft_std, float noise_std, float boost_fraction,
                                  float boost, int32_t* tokens, float* conf, uint8_t* in_step, uint32_t* device_round,
                                  void* workspace, size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* FEF_H */

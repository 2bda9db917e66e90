/*
 * CPU oracle for the FeF-DLLM speculative-verification step.
 *
 * TEST INFRASTRUCTURE ONLY. This is a plain, slow, single-threaded,
 * double-precision restatement of what the paper's decoding algorithm
 * computes per speculative window (Algorithm 2, inner verification loop;
 * the residual law of Eq. "residual_distribution_alg"; Section 3.2), and of
 * the LowConf selection of Algorithm 2.  It shares no code, header, table or
 * constant generator with the CUDA library and neither includes the other.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * All pointers are HOST pointers.  Layouts match the CUDA library's so the
 * same bytes can be given to both.
 *
 * Pins (tests/test_oracle_pins.py): Philox against the cuRAND host generator,
 * softmax against a float64 library softmax, acceptance probability
 * = sum_z min(pi, rho), emitted-token law = pi by exact enumeration and by
 * chi-square, p = q accepts everything, residual sums to one, mean committed
 * length = sum_l prod_{i<l} alpha_i (Theorem 2 when the alpha_i are equal),
 * LowConf against a library stable sort; draft sampling: frequencies against a library softmax
 * by chi-square, the temperature-0 limit against arg-max, invariance under a common shift.
 * Parity unpinned by the paper (readings fixed by this build only): the
 * confidence reported at temperature 0, tie order in LowConf, sentinel values
 * beyond the committed prefix.
 */
#ifndef FEF_ORACLE_H
#define FEF_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status values (numerically the same meaning as the library's, restated) */
enum {
    FEFO_OK = 0,
    FEFO_ERR_INVALID_ARG = 1,
    FEFO_ERR_DTYPE = 2,
    FEFO_ERR_NONFINITE = 7,
    FEFO_ERR_TOKEN_RANGE = 8
};

/* logit storage types (FEFO_F64: fef_oracle_spec_verify only; logits that come out of a
 * double-precision matrix product, see oracle/lmhead.py) */
enum { FEFO_F32 = 0, FEFO_BF16 = 1, FEFO_F64 = 2 };

/* Philox4x32-10 block function: out[4] = philox(ctr[4], key[2]). */
void fef_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* The uniform the verification step draws.
 * key = (low 32 bits of seed, high 32 bits of seed);
 * counter = ((stream << 30) | j, b, pos, step); the `lane`-th output word r
 * maps to u = ((r >> 9) + 0.5) * 2^-23, which lies strictly inside (0, 1). */
double fef_oracle_uniform(uint64_t seed, uint32_t stream, uint32_t j, uint32_t b,
                          uint32_t pos, uint32_t step, uint32_t lane);

/* Laws of ONE position (Section 3.2): pi = softmax(p_logits / T),
 * rho = softmax(q_logits / T), resid = [pi - rho]_+ / (1 - sum_z min(pi, rho))
 * (all zeros when that denominator is 0), *alpha = sum_z min(pi, rho).
 * T must be > 0.  Returns a status. */
int fef_oracle_row_laws(const void* p_logits, const void* q_logits, int V, int dtype,
                        float temperature, double* pi, double* rho, double* resid,
                        double* alpha);

/* One verification call over B independent windows of K positions
 * (Algorithm 2, the loop "for m = 1..b").
 *   draft_logits, target_logits : [B, K, ld] (ld >= V), dtype F32, BF16 or F64
 *   draft_tokens                : [B, K]
 *   row_len                     : [B] number of valid drafts (0..K), or NULL = K
 *   temperature                 : > 0 sampling; == 0 greedy (see the notes at the top of
 *                                 the .cpp); < 0 invalid
 *   batch_offset                : window b draws its random numbers as batch row
 *                                 batch_offset + b, so a slice of a larger batch can be
 *                                 checked on its own
 * Outputs (caller allocated):
 *   accept_len [B]    index of first rejected draft, or row_len if none; -1 on a data error
 *   tokens     [B, K] committed tokens (accepted drafts, then the corrected token); -1 beyond
 *   conf       [B, K] double; pi(committed token); -1 beyond
 *   accept_margin [B, K] (may be NULL) |u - pi(x)/rho(x)| of every acceptance test made, else +inf
 *   gumbel_gap    [B]    (may be NULL) best minus second-best Gumbel score of the
 *                        residual draw, +inf when no draw or a single candidate
 * Returns the largest status over the batch rows. */
int fef_oracle_spec_verify(const void* draft_logits, const void* target_logits,
                           const int32_t* draft_tokens, const int32_t* row_len,
                           int B, int K, int V, int64_t ld, int dtype,
                           float temperature, uint64_t seed, uint32_t step,
                           uint32_t batch_offset,
                           int32_t* accept_len, int32_t* tokens, double* conf,
                           double* accept_margin, double* gumbel_gap);

/* Draft-token sampling (Algorithm 2, "Sample draft tokens x~ ~ rho"; Section 3.2): for every
 * position i < row_len[b] one draw from rho = softmax(draft_logits[b,i,:] / T) by Gumbel-max,
 * arg-max_x { l_x / T - ln(-ln u_x) } over the entries with l_x > -inf, lowest x on exact ties;
 * u_x from stream 2: counter ((2 << 30) | (x >> 2), batch_offset + b, i, step), word x & 3.
 * T == 0: arg-max of the logits, no random numbers.
 *   draft_tokens [B, K]  the draws; -1 for i >= row_len[b] and for positions with a data error
 *   gumbel_gap   [B, K]  (may be NULL) best minus runner-up score, +inf if there is none
 * Returns the largest status (NaN, +inf or a row without a finite logit: FEFO_ERR_NONFINITE). */
int fef_oracle_draft_sample(const void* draft_logits, const int32_t* row_len, int B, int K, int V, int64_t ld,
                            int dtype, float temperature, uint64_t seed, uint32_t step, uint32_t batch_offset,
                            int32_t* draft_tokens, double* gumbel_gap);

/* LowConf_k (Algorithm 2): per batch row the k candidates (mask != 0) of lowest
 * confidence, ordered by (conf ascending, index ascending).
 *   conf [B, L] float, mask [B, L] uint8 -> positions [B, k] (-1 padded), count [B]. */
int fef_oracle_remask_select(const float* conf, const uint8_t* mask, int B, int L, int k,
                             int32_t* positions, int32_t* count);

#ifdef __cplusplus
}
#endif
#endif

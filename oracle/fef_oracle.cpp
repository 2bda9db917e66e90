// CPU oracle for the FeF-DLLM speculative-verification step.
// TEST INFRASTRUCTURE ONLY: see fef_oracle.h.  Plain C++17, double precision,
// one thread, no blocking or fusion: every function follows the paper's
// statement of the step it implements, in the paper's order.
//
// Readings this file fixes where the paper is silent (each is listed again in
// the design notes of the repository):
//  * both laws are softmax(logits / T) (the paper only says the temperature is
//    the baseline's, Appendix A);
//  * T == 0 is greedy: the laws are point masses at the arg-max (lowest index
//    on ties), a draft is accepted iff it equals arg-max of the target logits,
//    the replacement is that arg-max, no random number is consumed, and the
//    reported confidence is softmax(target logits, T = 1) of the committed
//    token (a point mass would make every confidence 1);
//  * rho(x) = 0: accept iff pi(x) > 0 (Theorem 1's proof uses
//    rho * min{1, pi/rho} = min{pi, rho});
//  * a rejection although sum_x [pi - rho]_+ == 0 (probability zero) commits
//    arg-max of pi;
//  * random numbers: Philox4x32-10, counter layout in fef_oracle.h; the
//    residual draw is Gumbel-max, arg-max over x with [pi - rho]_+ > 0 of
//    ln r_x - ln(-ln u_x), lowest x on exact ties.
#include "fef_oracle.h"

#include <algorithm>
#include <cmath>
#include <limits>
#include <vector>

namespace {

const double kInf = std::numeric_limits<double>::infinity();

// ---------------------------------------------------------------- logits ----
double load_logit(const void* base, int64_t index, int dtype) {
    if (dtype == FEFO_F64) {
        return static_cast<const double*>(base)[index];
    }
    if (dtype == FEFO_F32) {
        return (double)static_cast<const float*>(base)[index];
    }
    // bfloat16: the upper 16 bits of an IEEE binary32
    uint32_t bits = (uint32_t)static_cast<const uint16_t*>(base)[index] << 16;
    float f;
    static_assert(sizeof(f) == sizeof(bits), "float is 32 bits");
    std::copy(reinterpret_cast<const char*>(&bits), reinterpret_cast<const char*>(&bits) + 4,
              reinterpret_cast<char*>(&f));
    return (double)f;
}

std::vector<double> load_row(const void* base, int64_t offset, int V, int dtype) {
    std::vector<double> row((size_t)V);
    for (int v = 0; v < V; ++v) row[(size_t)v] = load_logit(base, offset + v, dtype);
    return row;
}

// A row is usable when it has no NaN, no +inf and at least one finite entry
// (-inf is legal: probability zero).
bool row_is_valid(const std::vector<double>& l) {
    bool any_finite = false;
    for (double x : l) {
        if (std::isnan(x)) return false;
        if (x == kInf) return false;
        if (std::isfinite(x)) any_finite = true;
    }
    return any_finite;
}

int argmax_lowest_index(const std::vector<double>& x) {
    int best = 0;
    for (int v = 1; v < (int)x.size(); ++v)
        if (x[(size_t)v] > x[(size_t)best]) best = v;
    return best;
}

// softmax(l / T), T > 0, by the textbook max-subtracted formula.
std::vector<double> softmax_T(const std::vector<double>& l, double T) {
    const size_t V = l.size();
    std::vector<double> z(V), p(V);
    for (size_t v = 0; v < V; ++v) z[v] = l[v] / T;
    double m = -kInf;
    for (size_t v = 0; v < V; ++v) m = std::max(m, z[v]);
    double S = 0.0;
    for (size_t v = 0; v < V; ++v) {
        p[v] = std::exp(z[v] - m);  // exp(-inf) = 0
        S += p[v];
    }
    for (size_t v = 0; v < V; ++v) p[v] /= S;
    return p;
}

// ---------------------------------------------------------------- Philox ----
// Philox4x32 with 10 rounds (Salmon et al., "Parallel random numbers: as easy
// as 1, 2, 3", 2011): each round multiplies words 0 and 2 by two fixed odd
// constants, mixes the high halves with words 1, 3 and the round key, and the
// key is bumped by two Weyl constants between rounds.
void philox_round(uint32_t c[4], const uint32_t k[2]) {
    const uint64_t prod0 = (uint64_t)0xD2511F53u * c[0];
    const uint64_t prod1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
    const uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
    const uint32_t n0 = hi1 ^ c[1] ^ k[0];
    const uint32_t n2 = hi0 ^ c[3] ^ k[1];
    c[0] = n0;
    c[1] = lo1;
    c[2] = n2;
    c[3] = lo0;
}

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k[0] += 0x9E3779B9u;
            k[1] += 0xBB67AE85u;
        }
        philox_round(c, k);
    }
    for (int i = 0; i < 4; ++i) out[i] = c[i];
}

double uniform_open01(uint64_t seed, uint32_t stream, uint32_t j, uint32_t b, uint32_t pos,
                      uint32_t step, uint32_t lane) {
    const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    const uint32_t ctr[4] = {(stream << 30) | j, b, pos, step};
    uint32_t r[4];
    philox4x32_10(ctr, key, r);
    // 23 random bits, centred in their bin: never 0, never 1, exact in binary32.
    return ((double)(r[lane] >> 9) + 0.5) * (1.0 / 8388608.0);
}

const uint32_t kStreamAccept = 0;    // one uniform per (b, pos, step)
const uint32_t kStreamResidual = 1;  // one uniform per (b, pos, step, vocabulary id)
const uint32_t kStreamDraft = 2;     // draft sampling: one uniform per (b, pos, step, vocabulary id)

// -------------------------------------------------------------- residual ----
// r_x = [pi(x) - rho(x)]_+   (numerator of the residual law)
std::vector<double> residual_numerator(const std::vector<double>& pi, const std::vector<double>& rho) {
    std::vector<double> r(pi.size());
    for (size_t x = 0; x < pi.size(); ++x) r[x] = std::max(0.0, pi[x] - rho[x]);
    return r;
}

// Z ~ r / sum(r) by Gumbel-max with one uniform per vocabulary id.
// Returns -1 when r is identically zero.  *gap = best score - runner-up score.
int sample_residual_gumbel(const std::vector<double>& r, uint64_t seed, uint32_t b, uint32_t pos,
                           uint32_t step, double* gap) {
    int best = -1;
    double best_score = -kInf, second_score = -kInf;
    for (int x = 0; x < (int)r.size(); ++x) {
        if (!(r[(size_t)x] > 0.0)) continue;
        const double u = uniform_open01(seed, kStreamResidual, (uint32_t)x >> 2, b, pos, step,
                                        (uint32_t)x & 3u);
        const double score = std::log(r[(size_t)x]) - std::log(-std::log(u));
        if (score > best_score) {  // strict: the lowest x keeps an exact tie
            second_score = best_score;
            best_score = score;
            best = x;
        } else if (score > second_score) {
            second_score = score;
        }
    }
    *gap = (best >= 0 && second_score > -kInf) ? best_score - second_score : kInf;
    return best;
}

// ------------------------------------------------------ one batch row (b) ----
struct RowOutputs {
    int32_t* accept_len;
    int32_t* tokens;        // [K]
    double* conf;           // [K]
    double* accept_margin;  // [K] or null
    double* gumbel_gap;     // scalar or null
};

void fill_sentinels(const RowOutputs& o, int K) {
    for (int i = 0; i < K; ++i) {
        o.tokens[i] = -1;
        o.conf[i] = -1.0;
        if (o.accept_margin) o.accept_margin[i] = kInf;
    }
    if (o.gumbel_gap) *o.gumbel_gap = kInf;
}

int verify_one_window(const void* q_base, const void* p_base, const int32_t* draft, int n, int K, int V,
                      int64_t ld, int dtype, double T, uint64_t seed, uint32_t b, uint32_t step,
                      const RowOutputs& o) {
    fill_sentinels(o, K);

    // data errors anywhere in the valid part of the window poison the window
    for (int i = 0; i < n; ++i)
        if (draft[i] < 0 || draft[i] >= V) {
            *o.accept_len = -1;
            return FEFO_ERR_TOKEN_RANGE;
        }
    for (int i = 0; i < n; ++i) {
        bool ok = row_is_valid(load_row(p_base, (int64_t)i * ld, V, dtype));
        if (T > 0.0) ok = ok && row_is_valid(load_row(q_base, (int64_t)i * ld, V, dtype));
        if (!ok) {
            *o.accept_len = -1;
            return FEFO_ERR_NONFINITE;
        }
    }

    int a = n;  // accept length if nothing is rejected
    for (int i = 0; i < n; ++i) {
        const std::vector<double> lp = load_row(p_base, (int64_t)i * ld, V, dtype);
        const int x = draft[i];

        if (T == 0.0) {
            // greedy reading: point masses; confidence from the T = 1 law
            const std::vector<double> pi1 = softmax_T(lp, 1.0);
            const int top = argmax_lowest_index(lp);
            if (x == top) {
                o.tokens[i] = x;
                o.conf[i] = pi1[(size_t)x];
                continue;
            }
            o.tokens[i] = top;
            o.conf[i] = pi1[(size_t)top];
            a = i;
            break;
        }

        const std::vector<double> lq = load_row(q_base, (int64_t)i * ld, V, dtype);
        const std::vector<double> pi = softmax_T(lp, T);   // target law
        const std::vector<double> rho = softmax_T(lq, T);  // draft law

        // acceptance test: u <= min{1, pi(x)/rho(x)}
        const double u = uniform_open01(seed, kStreamAccept, 0, b, (uint32_t)i, step, 0);
        bool accept;
        if (rho[(size_t)x] > 0.0) {
            const double ratio = pi[(size_t)x] / rho[(size_t)x];
            accept = (u <= std::min(1.0, ratio));
            if (o.accept_margin) o.accept_margin[i] = std::fabs(u - ratio);
        } else {
            accept = (pi[(size_t)x] > 0.0);
        }

        if (accept) {
            o.tokens[i] = x;
            o.conf[i] = pi[(size_t)x];
            continue;
        }

        // first rejection: draw the replacement from the residual law, commit it, stop
        const std::vector<double> r = residual_numerator(pi, rho);
        double gap = kInf;
        int Z = sample_residual_gumbel(r, seed, b, (uint32_t)i, step, &gap);
        if (Z < 0) Z = argmax_lowest_index(pi);  // residual mass is zero
        if (o.gumbel_gap) *o.gumbel_gap = gap;
        o.tokens[i] = Z;
        o.conf[i] = pi[(size_t)Z];
        a = i;
        break;
    }
    *o.accept_len = a;
    return FEFO_OK;
}

// ---------------------------------------------------------- draft sampling ----
// x~ ~ softmax(l / T) for one position (Algorithm 2, "Sample draft tokens"; Section 3.2) by
// Gumbel-max: arg-max over x of l_x / T - ln(-ln u_x), one uniform per vocabulary id, entries
// with l_x = -inf left out, lowest x on exact ties.  T == 0: arg-max of l (lowest index).
// Returns the token, -1 on a data error (NaN, +inf, or no finite logit).  *gap = best score
// minus runner-up score (in units of l / T; +inf with a single candidate or at T == 0).
int sample_draft_row(const void* row, int V, int dtype, double T, uint64_t seed, uint32_t b, uint32_t pos,
                     uint32_t step, double* gap, int* status) {
    int best = -1;
    double best_score = -kInf, second_score = -kInf;
    *gap = kInf;
    for (int x = 0; x < V; ++x) {
        const double l = load_logit(row, x, dtype);
        if (std::isnan(l) || l == kInf) {
            *status = FEFO_ERR_NONFINITE;
            return -1;
        }
        if (l == -kInf) continue;
        double score = l;
        if (T > 0.0) {
            const double u = uniform_open01(seed, kStreamDraft, (uint32_t)x >> 2, b, pos, step, (uint32_t)x & 3u);
            score = l / T - std::log(-std::log(u));
        }
        if (score > best_score) {  // strict: the lowest x keeps an exact tie
            second_score = best_score;
            best_score = score;
            best = x;
        } else if (score > second_score) {
            second_score = score;
        }
    }
    if (best < 0) {
        *status = FEFO_ERR_NONFINITE;
        return -1;
    }
    if (T > 0.0 && second_score > -kInf) *gap = best_score - second_score;
    return best;
}

}  // namespace

// ================================================================= C ABI ====
extern "C" {

void fef_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    philox4x32_10(ctr, key, out);
}

double fef_oracle_uniform(uint64_t seed, uint32_t stream, uint32_t j, uint32_t b, uint32_t pos,
                          uint32_t step, uint32_t lane) {
    return uniform_open01(seed, stream, j, b, pos, step, lane & 3u);
}

int fef_oracle_row_laws(const void* p_logits, const void* q_logits, int V, int dtype,
                        float temperature, double* pi_out, double* rho_out, double* resid_out,
                        double* alpha_out) {
    if (!p_logits || !q_logits || V < 1 || !(temperature > 0.0f)) return FEFO_ERR_INVALID_ARG;
    if (dtype != FEFO_F32 && dtype != FEFO_BF16) return FEFO_ERR_DTYPE;
    const std::vector<double> lp = load_row(p_logits, 0, V, dtype);
    const std::vector<double> lq = load_row(q_logits, 0, V, dtype);
    if (!row_is_valid(lp) || !row_is_valid(lq)) return FEFO_ERR_NONFINITE;
    const std::vector<double> pi = softmax_T(lp, (double)temperature);
    const std::vector<double> rho = softmax_T(lq, (double)temperature);
    const std::vector<double> r = residual_numerator(pi, rho);
    double alpha = 0.0;
    for (int x = 0; x < V; ++x) alpha += std::min(pi[(size_t)x], rho[(size_t)x]);
    const double denom = 1.0 - alpha;
    for (int x = 0; x < V; ++x) {
        if (pi_out) pi_out[x] = pi[(size_t)x];
        if (rho_out) rho_out[x] = rho[(size_t)x];
        if (resid_out) resid_out[x] = denom > 0.0 ? r[(size_t)x] / denom : 0.0;
    }
    if (alpha_out) *alpha_out = alpha;
    return FEFO_OK;
}

int fef_oracle_spec_verify(const void* draft_logits, const void* target_logits,
                           const int32_t* draft_tokens, const int32_t* row_len, int B, int K, int V,
                           int64_t ld, int dtype, float temperature, uint64_t seed, uint32_t step,
                           uint32_t batch_offset, int32_t* accept_len, int32_t* tokens, double* conf,
                           double* accept_margin, double* gumbel_gap) {
    if (!draft_logits || !target_logits || !draft_tokens || !accept_len || !tokens || !conf)
        return FEFO_ERR_INVALID_ARG;
    if (B < 1 || K < 1 || V < 1 || ld < V || !(temperature >= 0.0f)) return FEFO_ERR_INVALID_ARG;
    if (dtype != FEFO_F32 && dtype != FEFO_BF16 && dtype != FEFO_F64) return FEFO_ERR_DTYPE;
    if (row_len)
        for (int b = 0; b < B; ++b)
            if (row_len[b] < 0 || row_len[b] > K) return FEFO_ERR_INVALID_ARG;

    const int64_t elem = (dtype == FEFO_F64) ? 8 : (dtype == FEFO_F32) ? 4 : 2;
    int worst = FEFO_OK;
    for (int b = 0; b < B; ++b) {
        const int64_t window = (int64_t)b * K;
        const char* q = static_cast<const char*>(draft_logits) + window * ld * elem;
        const char* p = static_cast<const char*>(target_logits) + window * ld * elem;
        RowOutputs o;
        o.accept_len = accept_len + b;
        o.tokens = tokens + window;
        o.conf = conf + window;
        o.accept_margin = accept_margin ? accept_margin + window : nullptr;
        o.gumbel_gap = gumbel_gap ? gumbel_gap + b : nullptr;
        const int n = row_len ? row_len[b] : K;
        const int st = verify_one_window(q, p, draft_tokens + window, n, K, V, ld, dtype,
                                         (double)temperature, seed, batch_offset + (uint32_t)b, step, o);
        worst = std::max(worst, st);
    }
    return worst;
}

int fef_oracle_remask_select(const float* conf, const uint8_t* mask, int B, int L, int k,
                             int32_t* positions, int32_t* count) {
    if (!conf || !mask || !positions || !count || B < 1 || L < 1 || k < 0)
        return FEFO_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b) {
        const float* c = conf + (int64_t)b * L;
        std::vector<int32_t> cand;
        for (int i = 0; i < L; ++i)
            if (mask[(int64_t)b * L + i] != 0) cand.push_back(i);
        // ascending confidence; a stable sort keeps ascending index among equals;
        // NaN (not a valid confidence) sorts after every number
        std::stable_sort(cand.begin(), cand.end(), [c](int32_t i, int32_t j) {
            const bool ni = std::isnan(c[i]), nj = std::isnan(c[j]);
            if (ni || nj) return !ni && nj;
            return c[i] < c[j];
        });
        const int n = std::min<int>(k, (int)cand.size());
        count[b] = n;
        for (int t = 0; t < k; ++t) positions[(int64_t)b * k + t] = t < n ? cand[(size_t)t] : -1;
    }
    return FEFO_OK;
}

int fef_oracle_draft_sample(const void* draft_logits, const int32_t* row_len, int B, int K, int V, int64_t ld,
                            int dtype, float temperature, uint64_t seed, uint32_t step, uint32_t batch_offset,
                            int32_t* draft_tokens, double* gumbel_gap) {
    if (!draft_logits || !draft_tokens || B < 1 || K < 1 || V < 1 || ld < V) return FEFO_ERR_INVALID_ARG;
    if (dtype != FEFO_F32 && dtype != FEFO_BF16) return FEFO_ERR_DTYPE;
    if (!(temperature >= 0.0f)) return FEFO_ERR_INVALID_ARG;
    const int64_t esize = dtype == FEFO_F32 ? 4 : 2;
    int worst = FEFO_OK;
    for (int b = 0; b < B; ++b) {
        const int n = row_len ? std::min(std::max(row_len[b], 0), K) : K;
        for (int i = 0; i < K; ++i) {
            const int64_t row = (int64_t)b * K + i;
            draft_tokens[row] = -1;
            if (gumbel_gap) gumbel_gap[row] = kInf;
            if (i >= n) continue;
            int status = FEFO_OK;
            double gap = kInf;
            const char* base = (const char*)draft_logits + row * ld * esize;
            draft_tokens[row] = sample_draft_row(base, V, dtype, (double)temperature, seed, batch_offset + (uint32_t)b,
                                                 (uint32_t)i, step, &gap, &status);
            if (gumbel_gap) gumbel_gap[row] = gap;
            worst = std::max(worst, status);
        }
    }
    return worst;
}

}  // extern "C"

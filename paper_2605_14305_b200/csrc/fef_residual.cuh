// The residual draw Z ~ [pi - rho]_+ / (1 - sum min{pi, rho}) (the law defined before Algorithm 2) as
// device code shared by the verification kernels: bounds in binary32, the decision among the best
// candidates, the double-precision pass for draws the bounds cannot decide.
#pragma once

#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"
#include "fef_device_math.cuh"
#include "fef_verify_params.cuh"

namespace cg = cooperative_groups;

namespace fef {

constexpr int kResidualThreads = 256;
constexpr int kResidualWarps = kResidualThreads / 32;
constexpr int kCandidatesPerCta = 3;  // what a CTA leaves for the deciding warp
constexpr int kMaxClusterCtas = 8;    // up to this many CTAs per window they form a thread-block cluster
constexpr int kMaxResidualCtas = 2 * kResidualThreads / kCandidatesPerCta;  // reporting mode: two candidates per thread
constexpr int kResidualCtasPerSm = 2;  // resident CTAs the grid is sized for: 2 fat ones beat 4 (1.5 us per call) and 1

// Bound on the relative error of a law's normaliser as the streaming kernel delivers it (binary32
// partial sums of approximate exponentials; the largest error measured on a confidence is 1.1e-6,
// and that includes the rounding of the temperature scale).
constexpr double kNormRelErr = 2.0e-6;

__device__ __forceinline__ uint32_t pick_word(const uint4& w, int k) {
    return k == 0 ? w.x : k == 1 ? w.y : k == 2 ? w.z : w.w;
}

// The uniform of vocabulary id x (global id x + vocab_offset) in the residual draw of (b, pos).
static __device__ double residual_uniform(int x, uint32_t b, uint32_t pos, const VerifyParams& P) {
    const uint4 w = philox4x32_10(
        make_uint4((kStreamResidual << 30) | (static_cast<uint32_t>(x + P.vocab_offset) >> 2), b, pos, step_of(P)),
        make_uint2(static_cast<uint32_t>(P.seed), static_cast<uint32_t>(P.seed >> 32)));
    return uniform_from_word(pick_word(w, x & 3));
}

// Exact (double) Gumbel score ln r_x - ln(-ln u_x) of vocabulary id x with the given normalisers;
// -inf when r_x <= 0.
template <int DT>
__device__ double exact_score(int x, const char* prow, const char* qrow, double c, double kp, double kq,
                              uint32_t b, uint32_t pos, const VerifyParams& P) {
    const double lp = load_logit<DT>(prow, x);
    const double lq = load_logit<DT>(qrow, x);
    const double pi = exp2(lp * c - kp);
    const double rho = exp2(lq * c - kq);
    const double r = pi - rho;
    if (!(r > 0.0)) return -INFINITY;
    return log(r) - log(-log(residual_uniform(x, b, pos, P)));
}

struct ResidualShared {
    unsigned floor_bits;   // lower bound of the CTA's third-largest bound (bits of a float >= 0): the first estimate
    unsigned best3[3];     // three of the largest bounds offered so far by any thread of the CTA (bits): each slot
                           // holds the bound of a different id, so their minimum is such a lower bound too
    int last;              // this CTA is the window's last one to finish its share
    int exact;             // the deciding warp asks for the double-precision pass over the row
    float exact_floor;     // ... and gives it a lower bound of the row's largest true weight (0: none)
    Top3 top[kResidualWarps];
    Candidate cluster_cand[kMaxClusterCtas * kCandidatesPerCta];  // rank 0: what the cluster's CTAs found
    double red_a[kResidualWarps], red_b[kResidualWarps];
    int red_i[kResidualWarps];
};

// Block-wide arg-max of (score, lowest x).  Every thread gets the result.
static __device__ void block_argmax(double& score, int& x, ResidualShared& sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double os = __shfl_xor_sync(0xFFFFFFFFu, score, o);
        const int ox = __shfl_xor_sync(0xFFFFFFFFu, x, o);
        if (os > score || (os == score && ox < x)) {
            score = os;
            x = ox;
        }
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) {
        sh.red_a[warp] = score;
        sh.red_i[warp] = x;
    }
    __syncthreads();
    score = sh.red_a[0];
    x = sh.red_i[0];
    for (int w = 1; w < kResidualWarps; ++w)
        if (sh.red_a[w] > score || (sh.red_a[w] == score && sh.red_i[w] < x)) {
            score = sh.red_a[w];
            x = sh.red_i[w];
        }
}

// Block-wide sums of two doubles (fixed order: the same result in every thread and every run).
static __device__ void block_sum2(double& a, double& b, ResidualShared& sh) {
    a = warp_sum(a);
    b = warp_sum(b);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) {
        sh.red_a[warp] = a;
        sh.red_b[warp] = b;
    }
    __syncthreads();
    a = sh.red_a[0];
    b = sh.red_b[0];
    for (int w = 1; w < kResidualWarps; ++w) {
        a += sh.red_a[w];
        b += sh.red_b[w];
    }
}

// The residual draw of one row decided in double precision, normalisers included: both laws are
// summed again from the logits in double precision (the streaming kernel's binary32 sums only
// serve as the reference exponent), then arg-max_x { ln [pi - rho]_+ - ln(-ln u_x) }, lowest x on
// ties; if [pi - rho]_+ is zero everywhere, arg-max of the target logits.  `floor_w` is a lower bound
// of the row's largest true weight (0 = none known): ids whose binary32 upper bound cannot reach it
// are passed over after one multiply, as in the fast pass.  Whole CTA; every thread returns the
// same (Z, pi(Z)).  Slow (a pass of double-precision exponentials by one CTA): only for draws that
// the bounds of the fast pass cannot decide.
template <int DT>
__device__ void exact_row_draw(const VerifyParams& P, const char* prow, const char* qrow, uint32_t ub, uint32_t upos,
                               double kp_nom, double kq_nom, float slack, float floor_w, ResidualShared& sh, int& Z,
                               double& piZ) {
    const int V = P.geo.V;
    const double c = P.c_exact;
    // normalisers: sum_x 2^(l_x c - k_nominal) is within 1e-5 of one, so nothing can overflow
    double sp = 0.0, sq = 0.0;
    for (int x = threadIdx.x; x < V; x += kResidualThreads) {
        const double lp = load_logit<DT>(prow, x), lq = load_logit<DT>(qrow, x);
        if (lp > -INFINITY) sp += exp2(lp * c - kp_nom);
        if (lq > -INFINITY) sq += exp2(lq * c - kq_nom);
    }
    block_sum2(sp, sq, sh);
    const double kp = kp_nom + log2(sp), kq = kq_nom + log2(sq);
    const float kp32 = static_cast<float>(kp_nom), kq32 = static_cast<float>(kq_nom);

    PhiloxRow rng;
    rng.prepare(P.keys, ub, upos, step_of(P));
    double score = -INFINITY;
    int best = 0x7FFFFFFF;
    for (int pass = 0; pass < 2; ++pass) {
        // groups of four ids share a Philox call; a thread visits its ids in increasing order
        for (int x0 = 4 * static_cast<int>(threadIdx.x); x0 < V; x0 += 4 * kResidualThreads) {
            const uint4 w = rng.draw(P.keys, (kStreamResidual << 30) | (static_cast<uint32_t>(x0 + P.vocab_offset) >> 2));
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int x = x0 + k;
                if (x >= V) break;
                const float lpf = load_logit<DT>(prow, x), lqf = load_logit<DT>(qrow, x);
                const float ep = exp2_scaled<DT>(lpf, P.c_hi, P.c_lo, kp32);
                const float rs = fmaf(ep, slack, ep - exp2_scaled<DT>(lqf, P.c_hi, P.c_lo, kq32));
                const uint32_t word = pick_word(w, k);
                if (!(rs > floor_w * one_minus_uniform(word))) continue;
                const double pi = exp2(static_cast<double>(lpf) * c - kp);
                const double rho = lqf > -INFINITY ? exp2(static_cast<double>(lqf) * c - kq) : 0.0;
                const double r = pi - rho;
                if (!(r > 0.0)) continue;
                const double s = log(r) - log(-log(static_cast<double>(uniform_from_word(word))));
                if (s > score) {  // strict: the lowest index keeps a tie
                    score = s;
                    best = x;
                }
            }
        }
        block_argmax(score, best, sh);
        if (score > -INFINITY || floor_w == 0.f) break;
        floor_w = 0.f;  // (not expected: the floor belongs to an id of this row) once more without it
    }
    if (!(score > -INFINITY)) {
        // [pi - rho]_+ is identically zero: commit arg-max of pi (= arg-max of the target logits)
        score = -INFINITY;
        best = 0x7FFFFFFF;
        for (int x = threadIdx.x; x < V; x += kResidualThreads) {
            const double l = load_logit<DT>(prow, x);
            if (l > score) {
                score = l;
                best = x;
            }
        }
        block_argmax(score, best, sh);
    }
    Z = best;
    piZ = (best >= 0 && best < V) ? exp2(static_cast<double>(load_logit<DT>(prow, best)) * c - kp) : 0.0;
}

// Rare path of the residual pass, out of line so that the loop around it stays small: the id's
// bound ub = rs / (-ln u), rounded up (1.00003 is above the error of the approximate logarithm and
// division), offered to the thread's best three.
// The bound also enters the CTA's shared record of its largest bounds: three slots updated with
// atomic maxima, the smaller of (new, old) moving on to the next slot, so a value sits in one place
// only and every slot holds the bound of a different id.
static __device__ __noinline__ Top3 offer_bound(Top3 top, float rs, float t, int x, unsigned* best3) {
    const float ub = __fdividef(rs, neg_log_uniform(t)) * 1.00003f;
    top.offer(ub, x);
    unsigned v = __float_as_uint(ub);
    if (ub > 0.f && v > *reinterpret_cast<volatile unsigned*>(best3 + 2)) {
        unsigned old = atomicMax(best3, v);
        v = min(v, old);
        old = atomicMax(best3 + 1, v);
        v = min(v, old);
        atomicMax(best3 + 2, v);
    }
    return top;
}
// The lower bound of the CTA's third-largest bound that the shared record gives.
__device__ __forceinline__ float shared_floor(const unsigned* best3) {
    const volatile unsigned* b = best3;
    return __uint_as_float(min(min(b[0], b[1]), b[2]));
}

// The residual draw Z ~ [pi - rho]_+ / (1 - sum min{pi, rho}) of window b, rejected position `pos`,
// by Gumbel-max: arg-max_x { ln r_x - ln(-ln u_x) }, which is arg-max_x of w_x = r_x / (-ln u_x).
// This CTA covers share `part` of `parts` of the row; the window's last CTA to finish decides.
//
// Fast pass (binary32).  For every id an upper bound rs_x >= r_x that holds whatever the rounding of
// this pass and whatever the error of the two normalisers (each within kNormRelErr):
//     rs_x = (e_p - e_q) + slack * e_p,   e_p = 2^(l^p_x c - kp), e_q = 2^(l^q_x c - kq) in binary32.
// Since -ln u > 1 - u, an id with rs_x <= floor * (1 - u_x) has w_x < floor and is dropped after one
// multiply (floor = a lower bound of the CTA's third-largest bound so far); a warp vote keeps the few
// others out of the straight-line code.  Those get the bound ub_x = rs_x / (-ln u_x), rounded up, and
// each thread, warp and CTA keeps the three largest.
//
// Decision (one warp of the window's last CTA).  Of the row's three largest bounds, the ids x1, x2
// of the first two are evaluated in double precision: weight w = r / (-ln u) under the given
// normalisers and the interval [(r - 2 d pi) / (-ln u), (r + 2 d pi) / (-ln u)], d = kNormRelErr, that
// holds the weight under the exact normalisers.  Every other id's true weight is below the third
// bound.  If the larger of the two has its interval above the other's interval and above the third
// bound, it is the arg-max for every admissible value of the normalisers, hence the exact one:
// commit it.  Otherwise (two near-equal weights, or laws so close that pi - rho is lost in the
// normalisers' error) the row is redone by exact_row_draw.
//
// REPORT (vocabulary-parallel mode): the CTA's slice is one rank's share of the row and the ranks'
// best ids are compared afterwards by their scores under the shared normalisers, so the decision
// among this slice's candidates is taken on those scores (candidates within a band of the largest
// bound are scored in double precision) and reported instead of committed.
// prow, qrow: the target and draft logits of the rejected position; out_row: where tokens / conf go.
template <int DT, bool REPORT, bool CLUSTER>
__device__ void residual_draw(const VerifyParams& P, int b, int pos, double kp_d, double kq_d, const char* prow,
                              const char* qrow, int64_t out_row, int part, int parts, ResidualShared& sh) {
    constexpr int N = Elem<DT>::kPerVec;
    const Geometry& G = P.geo;
    const float kp = static_cast<float>(kp_d), kq = static_cast<float>(kq_d);
    const uint32_t ub = static_cast<uint32_t>(b), upos = static_cast<uint32_t>(pos);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // slack: relative to e_p.  Argument of the exponential: the narrowed normaliser (|k| 2^-24) and up
    // to two roundings of the multiply-adds (|l c - k| 2^-24 each, |l c - k| < 150 where e > 0), times
    // ln 2; ex2.approx: 2^-21; the subtraction: 2^-24; both laws.  Then the normalisers' own error
    // (reporting mode compares under the shared normalisers and leaves it out).
    const float rounding = (fabsf(kp) + fabsf(kq) + 600.f) * 4.2e-8f + 1.0e-6f;
    const float slack = REPORT ? rounding : rounding + static_cast<float>(2.0 * kNormRelErr);

    PhiloxRow rng;
    rng.prepare(P.keys, ub, upos, step_of(P));

    Top3 top;
    top.clear();
    float floor_w = 0.f;

    // ---- binary32 pass over this CTA's share of the row.  One vector pair (N ids of both laws) per
    //      thread and step; the loads of the next two steps are in flight while one is worked on.  The
    //      loop body is kept small (one copy, the rare path out of line): with several hundred
    //      instructions per step, a larger body stalls on instruction fetch.
    const int nvec = G.vec_elems / N;
    const int v_begin = static_cast<int>(static_cast<int64_t>(part) * nvec / parts);
    const int v_end = static_cast<int>(static_cast<int64_t>(part + 1) * nvec / parts);
    // a lane beyond the end works on -inf logits (rs = 0 never qualifies), so the warp stays whole
    constexpr uint32_t kMinusInf = DT == FEF_F32 ? 0xFF800000u : 0xFF80FF80u;
    auto fetch = [&](int v0, uint4& wp, uint4& wq) {
        const int vec = v0 + static_cast<int>(threadIdx.x);
        wp = wq = make_uint4(kMinusInf, kMinusInf, kMinusInf, kMinusInf);
        if (vec < v_end) {
            wp = ld_global_nc_v4(prow + static_cast<int64_t>(vec) * 16);
            wq = ld_global_nc_v4(qrow + static_cast<int64_t>(vec) * 16);
        }
    };
    // bounds rs and 1 - u of the N ids of one vector pair: straight-line, so that the Philox chains of
    // its groups of four ids and the exponentials overlap
    auto bounds = [&](int v0, const uint4& wp, const uint4& wq, float(&rs)[N], float(&t)[N]) {
        const int vec = v0 + static_cast<int>(threadIdx.x);
        float lp[N], lq[N];
        unpack<DT>(wp, lp);
        unpack<DT>(wq, lq);
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const float ep = exp2_scaled<DT>(lp[i], P.c_hi, P.c_lo, kp);
            rs[i] = fmaf(ep, slack, ep - exp2_scaled<DT>(lq[i], P.c_hi, P.c_lo, kq));
        }
#pragma unroll
        for (int g4 = 0; g4 < N / 4; ++g4) {
            const uint4 w = rng.draw(P.keys, (kStreamResidual << 30) |
                                                 (static_cast<uint32_t>(vec * N + 4 * g4 + P.vocab_offset) >> 2));
            t[4 * g4] = one_minus_uniform(w.x);
            t[4 * g4 + 1] = one_minus_uniform(w.y);
            t[4 * g4 + 2] = one_minus_uniform(w.z);
            t[4 * g4 + 3] = one_minus_uniform(w.w);
        }
    };

    // Two vector pairs per thread and step (their four Philox chains and 4 N exponentials overlap in the
    // straight-line part); the loads of the next step are in flight meanwhile.
    uint4 p0, q0, p1, q1, p2, q2, p3, q3;
    fetch(v_begin, p0, q0);
    fetch(v_begin + kResidualThreads, p1, q1);
    {
        // A first floor, so that the pass does not start with every id qualifying: the largest bound of
        // each lane's first vector pair; the third largest of the 32 belongs to a third distinct id, hence
        // is a lower bound of the CTA's third-largest bound.
        float rs[N], t[N];
        bounds(v_begin, p0, q0, rs, t);
        float m = 0.f;
#pragma unroll
        for (int i = 0; i < N; ++i)
            if (rs[i] > 0.f) m = fmaxf(m, __fdividef(rs[i], neg_log_uniform(t[i])));
        unsigned bits = __float_as_uint(m);
#pragma unroll
        for (int r = 0; r < 2; ++r) {  // drop the lanes holding the largest and the second largest
            const unsigned top_bits = __reduce_max_sync(0xFFFFFFFFu, bits);
            const unsigned holders = __ballot_sync(0xFFFFFFFFu, bits == top_bits);
            if (lane == __ffs(holders) - 1) bits = 0u;
        }
        floor_w = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, bits)) * 0.9999f;  // (the bounds above are not rounded up)
        if (lane == 0) atomicMax(&sh.floor_bits, __float_as_uint(floor_w));
    }
#pragma unroll 1
    for (int v0 = v_begin; v0 < v_end; v0 += 2 * kResidualThreads) {
        fetch(v0 + 2 * kResidualThreads, p2, q2);
        fetch(v0 + 3 * kResidualThreads, p3, q3);
        floor_w = fmaxf(fmaxf(floor_w, __uint_as_float(*reinterpret_cast<volatile unsigned*>(&sh.floor_bits))),
                        shared_floor(sh.best3));
        float rs[2 * N], t[2 * N];
        {
            float (&rs0)[N] = *reinterpret_cast<float(*)[N]>(rs);
            float (&t0)[N] = *reinterpret_cast<float(*)[N]>(t);
            float (&rs1)[N] = *reinterpret_cast<float(*)[N]>(rs + N);
            float (&t1)[N] = *reinterpret_cast<float(*)[N]>(t + N);
            bounds(v0, p0, q0, rs0, t0);
            bounds(v0 + kResidualThreads, p1, q1, rs1, t1);
        }
        unsigned qualify = 0u;
#pragma unroll
        for (int i = 0; i < 2 * N; ++i) qualify |= (rs[i] > floor_w * t[i]) ? (1u << i) : 0u;
        if (__any_sync(0xFFFFFFFFu, qualify != 0u)) {
#pragma unroll
            for (int i = 0; i < 2 * N; ++i)
                if (qualify & (1u << i))
                    top = offer_bound(top, rs[i], t[i],
                                      (v0 + (i / N) * kResidualThreads + static_cast<int>(threadIdx.x)) * N + (i % N),
                                      sh.best3);
            __syncwarp();
            floor_w = fmaxf(floor_w, shared_floor(sh.best3));  // (shared without a barrier)
        }
        p0 = p2;
        q0 = q2;
        p1 = p3;
        q1 = q3;
    }
    // tail elements (beyond the last whole vector) belong to part 0
    if (part == 0) {
        for (int x = G.vec_elems + threadIdx.x; x < G.V; x += kResidualThreads) {
            const float ep = exp2_scaled<DT>(load_logit<DT>(prow, x), P.c_hi, P.c_lo, kp);
            const float rsx = fmaf(ep, slack, ep - exp2_scaled<DT>(load_logit<DT>(qrow, x), P.c_hi, P.c_lo, kq));
            if (rsx > 0.f) {
                const uint4 w = rng.draw(P.keys, (kStreamResidual << 30) | (static_cast<uint32_t>(x + P.vocab_offset) >> 2));
                top = offer_bound(top, rsx, one_minus_uniform(pick_word(w, x & 3)), x, sh.best3);
            }
        }
    }

    // ---- CTA-wide best three (warp results meet in shared memory, warp 0 folds them), then the
    //      hand-over to the CTA that decides
    top.warp_merge();
    if (lane == 0) sh.top[warp] = top;
    __syncthreads();
    if (warp == 0) {
        Top3 all;
        all.clear();
        if (lane < kResidualWarps) all = sh.top[lane];
        all.warp_merge();
        if (lane == 0) {
            if constexpr (CLUSTER) {
                // the window's CTAs form one cluster: candidates go to rank 0's shared memory
                Candidate* out = cg::this_cluster().map_shared_rank(sh.cluster_cand, 0) + part * kCandidatesPerCta;
                out[0].w = all.w1;
                out[0].x = all.x1;
                out[1].w = all.w2;
                out[1].x = all.x2;
                out[2].w = all.w3;
                out[2].x = all.x3;
            } else {
                Candidate* out = P.candidates + (static_cast<int64_t>(b) * parts + part) * kCandidatesPerCta;
                out[0].w = all.w1;
                out[0].x = all.x1;
                out[1].w = all.w2;
                out[1].x = all.x2;
                out[2].w = all.w3;
                out[2].x = all.x3;
                __threadfence();
                const unsigned before = atomicAdd(&P.tasks[b].arrivals, 1u);
                sh.last = (before == static_cast<unsigned>(parts) - 1u);
            }
            sh.exact = 0;
        }
    }
    if constexpr (CLUSTER) {
        cg::this_cluster().sync();  // (every CTA of a window gets here or none does)
        if (part != 0) return;
    } else {
        __syncthreads();
        if (!sh.last) return;
        __threadfence();
    }

    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);
    const volatile Candidate* cand =
        CLUSTER ? sh.cluster_cand : P.candidates + static_cast<int64_t>(b) * parts * kCandidatesPerCta;
    const int ncand = parts * kCandidatesPerCta;

    if constexpr (!REPORT) {
        // ---- one warp decides
        if (warp == 0) {
            Top3 all;
            all.clear();
            if constexpr (CLUSTER) {  // at most 8 x 3 candidates, in shared memory
                for (int j = lane; j < ncand; j += 32) all.offer(cand[j].w, cand[j].x);
            } else {
                for (int j0 = 0; j0 < ncand; j0 += 8 * 32) {  // (all loads of a round first: they are volatile)
                    float cw[8];
                    int cx[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int j = j0 + k * 32 + lane;
                        cw[k] = j < ncand ? cand[j].w : 0.f;
                        cx[k] = j < ncand ? cand[j].x : 0x7FFFFFFF;  // (an empty slot, as Top3 keeps them)
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) all.offer(cw[k], cx[k]);
                }
            }
            all.warp_merge();
            // lanes 0 and 1: the ids of the two largest bounds.  First in binary32 with the same bounds as
            // the pass (a few hundred cycles); only when those do not separate them, in double precision.
            const int xe = lane == 0 ? all.x1 : all.x2;
            const float we = lane == 0 ? all.w1 : all.w2;
            const bool have = lane < 2 && we > 0.f && xe >= 0 && xe < G.V;
            float lpf = 0.f, lqf = 0.f, lb32 = -1.f, ub32 = 0.f;
            uint32_t word = 0u;
            if (have) {
                lpf = load_logit<DT>(prow, xe);
                lqf = load_logit<DT>(qrow, xe);
                word = pick_word(rng.draw(P.keys, (kStreamResidual << 30) | (static_cast<uint32_t>(xe + P.vocab_offset) >> 2)),
                                 xe & 3);
                const float ep = exp2_scaled<DT>(lpf, P.c_hi, P.c_lo, kp);
                const float r32 = ep - exp2_scaled<DT>(lqf, P.c_hi, P.c_lo, kq);
                const float e32 = neg_log_uniform(one_minus_uniform(word));
                ub32 = __fdividef(fmaf(ep, slack, r32), e32) * 1.00003f;
                lb32 = __fdividef(fmaf(ep, -slack, r32), e32) * 0.99997f;
            }
            const float lb_a = __shfl_sync(0xFFFFFFFFu, lb32, 0), lb_b = __shfl_sync(0xFFFFFFFFu, lb32, 1);
            const float ub_a = __shfl_sync(0xFFFFFFFFu, ub32, 0), ub_b = __shfl_sync(0xFFFFFFFFu, ub32, 1);
            const bool first32 = lb_a >= lb_b;
            const float lo32 = first32 ? lb_a : lb_b, hi32 = first32 ? ub_b : ub_a;
            if (lo32 > 1e-37f && lo32 > hi32 && lo32 > all.w3) {  // (the same in every lane)
                if (lane == (first32 ? 0 : 1)) {
                    P.tokens[out_row] = xe;
                    P.conf[out_row] = static_cast<float>(exp2(static_cast<double>(lpf) * c - kp_d));
                }
            } else {
                double wn = -1.0, lo = -1.0, hi = 0.0, pi = 0.0;
                if (have) {
                    pi = exp2(static_cast<double>(lpf) * c - kp_d);
                    const double r = pi - exp2(static_cast<double>(lqf) * c - kq_d);
                    const double e = -log(static_cast<double>(uniform_from_word(word)));
                    wn = r / e;
                    lo = (r - 2.0 * kNormRelErr * pi) / e * (1.0 - 1e-12);
                    hi = (r + 2.0 * kNormRelErr * pi) / e * (1.0 + 1e-12);
                }
                const double wn2 = __shfl_sync(0xFFFFFFFFu, wn, 1), lo2 = __shfl_sync(0xFFFFFFFFu, lo, 1);
                const double hi2 = __shfl_sync(0xFFFFFFFFu, hi, 1), pi2 = __shfl_sync(0xFFFFFFFFu, pi, 1);
                if (lane == 0) {
                    const bool first = wn >= wn2;
                    const double lo_w = first ? lo : lo2, hi_o = first ? hi2 : hi;
                    if (lo_w > 1e-300 && lo_w > hi_o && lo_w > static_cast<double>(all.w3)) {
                        P.tokens[out_row] = first ? all.x1 : all.x2;
                        P.conf[out_row] = static_cast<float>(first ? pi : pi2);
                    } else {
                        sh.exact = 1;
                        // a lower bound of the largest true weight, rounded down, for the double-precision pass
                        const double lb = fmax(fmax(lo, lo2), 0.0);
                        sh.exact_floor = lb > 1e-30 ? __double2float_rd(lb) * (1.0f - 1e-6f) : 0.f;
                    }
                }
            }
        }
        __syncthreads();
        if (!sh.exact) return;
        int Z;
        double piZ;
        exact_row_draw<DT>(P, prow, qrow, ub, upos, kp_d, kq_d, slack, sh.exact_floor, sh, Z, piZ);
        if (threadIdx.x == 0) {
            if (Z < 0 || Z >= G.V) {  // no finite target logit: the scan has reported such a row already
                P.tokens[out_row] = -1;
                P.conf[out_row] = -1.f;
                report(P.status, FEF_ERR_NONFINITE);
            } else {
                P.tokens[out_row] = Z;
                P.conf[out_row] = static_cast<float>(piZ);
            }
        }
    } else {
        // ---- this rank's best id by its score under the shared normalisers: candidates whose bound
        //      is within a band of the largest are scored in double precision
        // (at most kMaxResidualCtas * kCandidatesPerCta = 2 * kResidualThreads candidates: two per thread)
        float w[2] = {0.f, 0.f};
        int x[2] = {0x7FFFFFFF, 0x7FFFFFFF};
        double wbest = 0.0;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int j = static_cast<int>(threadIdx.x) + k * kResidualThreads;
            if (j < ncand) {
                w[k] = cand[j].w;
                x[k] = cand[j].x;
            }
            wbest = fmax(wbest, static_cast<double>(w[k]));
        }
        int dummy = 0;
        block_argmax(wbest, dummy, sh);
        const double band = fmax(1.0 / 512.0, 64.0 * static_cast<double>(slack));
        double score = -INFINITY;
        int Z = 0x7FFFFFFF;
#pragma unroll
        for (int k = 0; k < 2; ++k)
            if (w[k] > 0.f && static_cast<double>(w[k]) >= wbest * (1.0 - band)) {
                const double sc = exact_score<DT>(x[k], prow, qrow, c, kp_d, kq_d, ub, upos, P);
                if (sc > score || (sc == score && sc > -INFINITY && x[k] < Z)) {
                    score = sc;
                    Z = x[k];
                }
            }
        block_argmax(score, Z, sh);
        bool have_score = true;
        if (!(score > -INFINITY)) {
            // nothing with a positive residual among the candidates: go over the slice in double precision
            score = -INFINITY;
            Z = 0x7FFFFFFF;
            for (int xx = threadIdx.x; xx < G.V; xx += kResidualThreads) {
                const double s = exact_score<DT>(xx, prow, qrow, c, kp_d, kq_d, ub, upos, P);
                if (s > score) {  // increasing xx: the lowest index keeps a tie
                    score = s;
                    Z = xx;
                }
            }
            block_argmax(score, Z, sh);
            if (!(score > -INFINITY)) {
                // [pi - rho]_+ is zero on the slice: report the arg-max of the target logits
                have_score = false;
                score = -INFINITY;
                Z = 0x7FFFFFFF;
                for (int xx = threadIdx.x; xx < G.V; xx += kResidualThreads) {
                    const double l = load_logit<DT>(prow, xx);
                    if (l > score) {
                        score = l;
                        Z = xx;
                    }
                }
                block_argmax(score, Z, sh);
            }
        }
        if (threadIdx.x == 0) {
            const bool none = Z < 0 || Z >= G.V;  // the slice holds no finite target logit
            VpCandidate out;
            out.score = (have_score && !none) ? score : -INFINITY;
            out.lp = none ? -INFINITY : load_logit<DT>(prow, Z);
            out.index = none ? 0x7FFFFFFF : Z + P.vocab_offset;
            P.vp_out[b] = out;
        }
    }
}

}  // namespace fef

// fef_draft_sample: the draft tokens of a speculative window (Algorithm 2, "Sample draft tokens
// x~ ~ rho"; Section 3.2), one Gumbel-max draw per position from rho = softmax(draft logits / T).
//
// One kernel.  A row of draft logits is shared by `parts` CTAs (one CTA per row when there are
// many rows).  A thread reads its 16-byte vectors directly (the kernel is bound by the Philox
// arithmetic, not by memory), keeps the running sum of 2^(l c - ref) - which gives the draft
// law's normaliser as a by-product and makes bad data show - and the best two Gumbel keys
// l c - log2(-ln u) in binary32.  Nearly every id ends after one compare: since -ln u > 1 - u, an
// id can only beat the floor (a lower bound of the CTA's second-best key) if
// 1 - u < 2^(l c - floor), and 2^(l c - ref) is there already.  The last CTA of a row re-scores
// the finalists in double precision, so the token is the exact arg-max the definition asks for.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"
#include "fef_device_math.cuh"

namespace fef {

constexpr int kDraftThreads = 256;
constexpr int kDraftMaxParts = 64;      // CTAs per row at most (the last one looks at 2 keys per part)
constexpr uint32_t kStreamDraft = 2u;   // Philox stream of the draft draws
constexpr float kKeyBand = 1.0f / 1024.0f;  // binary32 keys this close to the best one are re-scored exactly

struct __align__(16) DraftPart {  // what one CTA leaves for the row's last CTA
    float ref, sum;   // sum of 2^(l c - ref) over the part (NaN when the data is bad)
    float k1, k2;     // best two keys (-inf when empty)
    int x1, x2;       // their vocabulary ids
    float tref, tsum; // the same sum over the target row's part, when the call also reduces the target rows
};

struct DraftParams {
    const char* logits;
    const char* target;  // target logits of the same shape, or null: their rows are summed in the same pass
    const int32_t* row_len;
    int B, K, V;
    int vec_elems;       // elements covered by whole 16-byte vectors; the rest is the row's tail
    int parts;           // CTAs per row
    int64_t ld_bytes;
    float c_hi, c_lo;    // log2(e)/T split in two binary32 numbers (c_lo = 0 for bfloat16)
    uint64_t seed;
    uint32_t step;
    const uint32_t* round; // device word added to `step` when the kernel runs, or null
    PhiloxKeys keys;     // round keys of `seed`
    int32_t* tokens;     // [B, K]
    double* log2_norm;   // [B, K] or null
    double* target_log2_norm;  // [B, K]: log2 normaliser of the target law (with `target`)
    DraftPart* part_out; // [B*K][parts]
    unsigned* arrivals;  // [B*K], cleared by the host call
    int32_t* status;
};

// Best two (key, lowest id); keys may be negative, empty = -inf.
struct BestTwo {
    float k1, k2;
    int x1, x2;
    __device__ __forceinline__ void clear() {
        k1 = k2 = -INFINITY;
        x1 = x2 = 0x7FFFFFFF;
    }
    __device__ __forceinline__ void offer(float k, int x) {
        if (better(k, x, k1, x1)) {
            k2 = k1;
            x2 = x1;
            k1 = k;
            x1 = x;
        } else if (better(k, x, k2, x2)) {
            k2 = k;
            x2 = x;
        }
    }
    __device__ __forceinline__ void warp_merge() {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ok1 = __shfl_xor_sync(0xFFFFFFFFu, k1, o), ok2 = __shfl_xor_sync(0xFFFFFFFFu, k2, o);
            const int ox1 = __shfl_xor_sync(0xFFFFFFFFu, x1, o), ox2 = __shfl_xor_sync(0xFFFFFFFFu, x2, o);
            offer(ok1, ox1);
            offer(ok2, ox2);
        }
    }
};

__device__ __forceinline__ uint32_t step_of(const DraftParams& P) {
    return P.step + (P.round ? __ldg(P.round) : 0u);
}

// Rare path of the draft pass, out of line so that the loop around it stays small: the id's key
// l c - log2(-ln u) in binary32, offered to the thread's best two and to the CTA's shared record of
// its largest keys (two slots updated with atomic maxima, the smaller of (new, old) moving on to the
// second slot, so a value sits in one place only and the slots hold keys of different ids).
static __device__ __noinline__ BestTwo offer_key(BestTwo top, float lc, uint32_t word, int x, int* best2) {
    const float key = lc - lg2_approx(neg_log_uniform(one_minus_uniform(word)));
    top.offer(key, x);
    int v = float_order(key);
    if (v > *reinterpret_cast<volatile int*>(best2 + 1)) {
        const int old = atomicMax(best2, v);
        v = min(v, old);
        atomicMax(best2 + 1, v);
    }
    return top;
}
// The lower bound of the CTA's second-best key that the shared record gives.
__device__ __forceinline__ float shared_floor2(const int* best2) {
    const volatile int* b = best2;
    return float_unorder(min(b[0], b[1]));
}

// Exact (double) key l / T - ln(-ln u) of vocabulary id x, in units of log2: l c - log2(-ln u).
template <int DT>
__device__ double exact_key(int x, const char* row, double c, uint32_t b, uint32_t pos, const DraftParams& P) {
    const double l = load_logit<DT>(row, x);
    if (!(l > -INFINITY)) return -INFINITY;
    const uint4 w = philox4x32_10(make_uint4((kStreamDraft << 30) | (static_cast<uint32_t>(x) >> 2), b, pos, step_of(P)),
                                  make_uint2(static_cast<uint32_t>(P.seed), static_cast<uint32_t>(P.seed >> 32)));
    const uint32_t word = (x & 3) == 0 ? w.x : (x & 3) == 1 ? w.y : (x & 3) == 2 ? w.z : w.w;
    const double u = uniform_from_word(word);
    return l * c - log2(-log(u));
}

template <int DT, bool GREEDY, bool WITH_TARGET>
__global__ void __launch_bounds__(kDraftThreads, WITH_TARGET ? 3 : 4) draft_kernel(const __grid_constant__ DraftParams P) {
    constexpr int N = Elem<DT>::kPerVec;
    const int parts = P.parts;
    const int64_t row = blockIdx.x / parts;
    const int part = static_cast<int>(blockIdx.x - row * parts);
    const int b = static_cast<int>(row / P.K), i = static_cast<int>(row - static_cast<int64_t>(b) * P.K);
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), P.K) : P.K;
    if (i >= n) {  // uniform over the CTA
        if (part == 0 && threadIdx.x == 0) {
            P.tokens[row] = -1;
            if (P.log2_norm) P.log2_norm[row] = 0.0;
            if (WITH_TARGET) P.target_log2_norm[row] = 0.0;
        }
        return;
    }
    const char* lrow = P.logits + row * P.ld_bytes;
    const char* trow = WITH_TARGET ? P.target + row * P.ld_bytes : nullptr;
    const uint32_t ub = static_cast<uint32_t>(b), upos = static_cast<uint32_t>(i);
    PhiloxRow rng;
    rng.prepare(P.keys, ub, upos, step_of(P));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    RowState st, stt;  // stt: the target row's sum (WITH_TARGET)
    st.reset();
    stt.reset();
    BestTwo top;
    top.clear();
    // Two of the largest keys any thread of the CTA has offered so far (ordered integers, see
    // offer_key): their minimum is a lower bound of the CTA's second-best key, the floor below which
    // an id cannot matter.  A stale value is only less sharp.
    __shared__ int s_best2[2];
    if (threadIdx.x == 0) s_best2[0] = s_best2[1] = float_order(-INFINITY);
    __syncthreads();
    float floor_k = -INFINITY;

    const int nvec = P.vec_elems / N;
    const int v_begin = static_cast<int>(static_cast<int64_t>(part) * nvec / parts);
    const int v_end = static_cast<int>(static_cast<int64_t>(part + 1) * nvec / parts);
    // a lane beyond the end works on -inf logits (they never qualify), so the warp stays whole
    constexpr uint32_t kMinusInf = DT == FEF_F32 ? 0xFF800000u : 0xFF80FF80u;
    auto fetch = [&](int v0, uint4& w) {
        const int vec = v0 + static_cast<int>(threadIdx.x);
        w = make_uint4(kMinusInf, kMinusInf, kMinusInf, kMinusInf);
        if (vec < v_end) w = ld_global_nc_v4(lrow + static_cast<int64_t>(vec) * 16);
    };
    // One vector per thread and step, the loads of the next two steps in flight; the loop body is kept
    // small (one copy, the rare path out of line): a larger one stalls on instruction fetch.
    auto fetch_target = [&](int v0, uint4& w) {
        const int vec = v0 + static_cast<int>(threadIdx.x);
        w = make_uint4(kMinusInf, kMinusInf, kMinusInf, kMinusInf);
        if (vec < v_end) w = ld_global_nc_v4(trow + static_cast<int64_t>(vec) * 16);
    };
    uint4 w0, w1, w2;
    uint4 t0, t1, t2;
    fetch(v_begin, w0);
    fetch(v_begin + kDraftThreads, w1);
    if constexpr (WITH_TARGET) {
        fetch_target(v_begin, t0);
        fetch_target(v_begin + kDraftThreads, t1);
    }
#pragma unroll 1
    for (int v0 = v_begin; v0 < v_end; v0 += kDraftThreads) {
        fetch(v0 + 2 * kDraftThreads, w2);
        if constexpr (WITH_TARGET) {
            // the target row's share of the same pass: sum of 2^(l c - ref), as in the streaming kernel
            fetch_target(v0 + 2 * kDraftThreads, t2);
            if (v0 + static_cast<int>(threadIdx.x) < v_end) {
                if (stt.ref == kNoReference) stt.ref = first_reference<DT>(t0, P.c_hi, P.c_lo);
                float lt[N];
                unpack<DT>(t0, lt);
                float ts = 0.f;
#pragma unroll
                for (int t = 0; t < N; ++t) ts += exp2_scaled<DT>(lt[t], P.c_hi, P.c_lo, stt.ref);
                if (ts <= kRescaleAbove)
                    stt.sum += ts;
                else
                    absorb_vector<DT, false>(t0, 0, P.c_hi, P.c_lo, stt);
            }
            t0 = t1;
            t1 = t2;
        }
        const int vec = v0 + static_cast<int>(threadIdx.x);
        floor_k = fmaxf(floor_k, shared_floor2(s_best2));
        float l[N], e[N];
        unpack<DT>(w0, l);
        if (st.ref == kNoReference) st.ref = first_reference<DT>(w0, P.c_hi, P.c_lo);
        const float ref_used = st.ref;  // the slow way below may move st.ref; e[] stays relative to this one
#pragma unroll
        for (int t = 0; t < N; ++t) e[t] = exp2_scaled<DT>(l[t], P.c_hi, P.c_lo, ref_used);
        float vs;
        if constexpr (N == 8)
            vs = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
        else
            vs = (e[0] + e[1]) + (e[2] + e[3]);
        if (vs <= kRescaleAbove)
            st.sum += vs;
        else  // reference missing or far too low, or bad data: the slow way moves it
            absorb_vector<DT, false>(w0, 0, P.c_hi, P.c_lo, st);
        if constexpr (GREEDY) {
            // temperature 0: the key is the logit itself
#pragma unroll
            for (int t = 0; t < N; ++t)
                if (l[t] > top.k2) top.offer(l[t], vec * N + t);
        } else {
            // an id can reach the floor only if 1 - u < 2^(l c - floor) = e * 2^(ref - floor)
            // (the factor keeps an id whose key ties the floor within binary32 rounding).
            // 1 - u < e * scale, with u's 23 bits = word >> 9, reads word > 2^32 - 256 - e * scale * 2^32:
            // one multiply-add, one conversion (negative and NaN give 0) and one integer compare per
            // id.  The constant 2^32 - 1024 and the factor leave room for every rounding, so no id
            // is missed; an id let through in error (-inf logits while there is no floor yet, one
            // word in 2^22 otherwise) is sorted out by the exact arithmetic at the end.
            const float s32 = 1.00001f * ex2_approx(ref_used - floor_k) * 4294967296.0f * 1.00002f;
            uint32_t word[N];
#pragma unroll
            for (int g4 = 0; g4 < N / 4; ++g4) {
                const uint4 r = rng.draw(P.keys, (kStreamDraft << 30) | (static_cast<uint32_t>(vec * N + 4 * g4) >> 2));
                word[4 * g4] = r.x;
                word[4 * g4 + 1] = r.y;
                word[4 * g4 + 2] = r.z;
                word[4 * g4 + 3] = r.w;
            }
            unsigned qualify = 0u;
#pragma unroll
            for (int t = 0; t < N; ++t)
                qualify |= (word[t] >= __float2uint_rz(fmaf(-e[t], s32, 4294966272.0f))) ? (1u << t) : 0u;
            if (__any_sync(0xFFFFFFFFu, qualify != 0u)) {  // the vote keeps this out of the straight line
#pragma unroll
                for (int t = 0; t < N; ++t)
                    if ((qualify & (1u << t)) && l[t] > -INFINITY) {
                        float lc = l[t] * P.c_hi;
                        if constexpr (Elem<DT>::kSplitScale) lc = fmaf(l[t], P.c_lo, lc);
                        top = offer_key(top, lc, word[t], vec * N + t, s_best2);
                    }
                __syncwarp();
                floor_k = fmaxf(floor_k, shared_floor2(s_best2));
            }
        }
        w0 = w1;
        w1 = w2;
    }

    // ---- CTA-wide: sum and best two
    const float M = float_unorder(__reduce_max_sync(0xFFFFFFFFu, float_order(st.ref)));
    float ssum = st.sum * ex2_approx(st.ref - M);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ssum += __shfl_xor_sync(0xFFFFFFFFu, ssum, o);
    float tM = 0.f, tsum = 0.f;
    if constexpr (WITH_TARGET) {
        tM = float_unorder(__reduce_max_sync(0xFFFFFFFFu, float_order(stt.ref)));
        tsum = stt.sum * ex2_approx(stt.ref - tM);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tsum += __shfl_xor_sync(0xFFFFFFFFu, tsum, o);
    }
    top.warp_merge();
    __shared__ DraftPart s_part[kDraftThreads / 32];
    __shared__ int s_last;
    if (lane == 0) {
        DraftPart d;
        d.ref = M;
        d.sum = ssum;
        d.k1 = top.k1;
        d.k2 = top.k2;
        d.x1 = top.x1;
        d.x2 = top.x2;
        d.tref = tM;
        d.tsum = tsum;
        s_part[warp] = d;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        DraftPart all = s_part[0];
        BestTwo bt;
        bt.k1 = all.k1;
        bt.k2 = all.k2;
        bt.x1 = all.x1;
        bt.x2 = all.x2;
        for (int wv = 1; wv < kDraftThreads / 32; ++wv) {
            const DraftPart o = s_part[wv];
            const float Mn = fmaxf(all.ref, o.ref);
            all.sum = all.sum * ex2_approx(all.ref - Mn) + o.sum * ex2_approx(o.ref - Mn);
            all.ref = Mn;
            if constexpr (WITH_TARGET) {
                const float Tn = fmaxf(all.tref, o.tref);
                all.tsum = all.tsum * ex2_approx(all.tref - Tn) + o.tsum * ex2_approx(o.tref - Tn);
                all.tref = Tn;
            }
            bt.offer(o.k1, o.x1);
            bt.offer(o.k2, o.x2);
        }
        all.k1 = bt.k1;
        all.k2 = bt.k2;
        all.x1 = bt.x1;
        all.x2 = bt.x2;
        P.part_out[row * parts + part] = all;
        unsigned before = static_cast<unsigned>(parts) - 1u;
        if (parts > 1) {
            __threadfence();
            before = atomicAdd(P.arrivals + row, 1u);
        }
        s_last = (before == static_cast<unsigned>(parts) - 1u);
    }
    __syncthreads();
    if (!s_last) return;
    if (parts > 1) __threadfence();

    // ---- the row's last CTA: normaliser and exact decision (first warp)
    if (warp != 0) return;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);
    const volatile DraftPart* po = P.part_out + row * parts;
    double m = -INFINITY, sacc = 0.0;
    int bad = 0;
    float kbest = -INFINITY;
    for (int p = lane; p < parts; p += 32) {
        const float pref = po[p].ref, psum = po[p].sum;
        if (!(psum >= 0.f) || psum == INFINITY) bad = 1;
        if (psum > 0.f) {
            const double pm = pref, ps = psum;
            if (pm > m) {
                sacc = sacc * exp2(m - pm) + ps;
                m = pm;
            } else {
                sacc += ps * exp2(pm - m);
            }
        }
        kbest = fmaxf(kbest, po[p].k1);
    }
    // tail elements (beyond the last whole vector): sum and exact keys
    double score = -INFINITY;
    int Z = 0x7FFFFFFF;
    for (int x = P.vec_elems + lane; x < P.V; x += 32) {
        const float l = load_logit<DT>(lrow, x);
        if (l != l || l == INFINITY) {
            bad = 1;
        } else if (l > -INFINITY) {
            const double pm = static_cast<double>(l) * c;
            if (pm > m) {
                sacc = sacc * exp2(m - pm) + 1.0;
                m = pm;
            } else {
                sacc += exp2(pm - m);
            }
            const double s = GREEDY ? static_cast<double>(l) : exact_key<DT>(x, lrow, c, ub, upos, P);
            if (s > score || (s == score && x < Z)) {
                score = s;
                Z = x;
            }
        }
    }
    double Mw = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Mw = fmax(Mw, __shfl_xor_sync(0xFFFFFFFFu, Mw, o));
    double S = m > -INFINITY ? sacc * exp2(m - Mw) : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(0xFFFFFFFFu, S, o);
    bad = __any_sync(0xFFFFFFFFu, bad) || !(S > 0.0) || !(S < INFINITY);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kbest = fmaxf(kbest, __shfl_xor_sync(0xFFFFFFFFu, kbest, o));

    // finalists: every part's two keys within the band of the best binary32 key
    for (int k = lane; k < 2 * parts; k += 32) {
        const float kk = (k & 1) ? po[k >> 1].k2 : po[k >> 1].k1;
        const int x = (k & 1) ? po[k >> 1].x2 : po[k >> 1].x1;
        if (kk > -INFINITY && kk >= kbest - kKeyBand) {
            const double s = GREEDY ? static_cast<double>(kk) : exact_key<DT>(x, lrow, c, ub, upos, P);
            if (s > score || (s == score && x < Z)) {
                score = s;
                Z = x;
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double os = __shfl_xor_sync(0xFFFFFFFFu, score, o);
        const int oz = __shfl_xor_sync(0xFFFFFFFFu, Z, o);
        if (os > score || (os == score && oz < Z)) {
            score = os;
            Z = oz;
        }
    }
    if constexpr (WITH_TARGET) {
        // the target law's normaliser from the parts' sums and the row's tail elements (NaN on bad data:
        // the verification that takes it reports the window)
        double tm = -INFINITY, ts = 0.0;
        int tbad = 0;
        for (int p = lane; p < parts; p += 32) {
            const float pref = po[p].tref, psum = po[p].tsum;
            if (!(psum >= 0.f) || psum == INFINITY) tbad = 1;
            if (psum > 0.f) {
                const double pm = pref, ps = psum;
                if (pm > tm) {
                    ts = tm > -INFINITY ? ts * exp2(tm - pm) + ps : ps;
                    tm = pm;
                } else {
                    ts += ps * exp2(pm - tm);
                }
            }
        }
        for (int x = P.vec_elems + lane; x < P.V; x += 32) {
            const float l = load_logit<DT>(trow, x);
            if (l != l || l == INFINITY) {
                tbad = 1;
            } else if (l > -INFINITY) {
                const double pm = static_cast<double>(l) * c;
                if (pm > tm) {
                    ts = tm > -INFINITY ? ts * exp2(tm - pm) + 1.0 : 1.0;
                    tm = pm;
                } else {
                    ts += exp2(pm - tm);
                }
            }
        }
        const double tMw = warp_max(tm);
        const double tS = warp_sum(tm > -INFINITY ? ts * exp2(tm - tMw) : 0.0);
        tbad = __any_sync(0xFFFFFFFFu, tbad) || !(tS > 0.0) || !(tS < INFINITY);
        if (lane == 0) P.target_log2_norm[row] = tbad ? __longlong_as_double(0x7FF8000000000000ll) : tMw + log2(tS);
    }
    if (lane == 0) {
        const bool ok = !bad && score > -INFINITY;
        P.tokens[row] = ok ? Z : -1;
        if (P.log2_norm) P.log2_norm[row] = ok ? Mw + log2(S) : 0.0;
        if (!ok) report(P.status, FEF_ERR_NONFINITE);
    }
}

static int draft_parts(int B, int K, int V, fef_dtype dt, int sm_count) {
    const int64_t rows = static_cast<int64_t>(B) * K;
    const int nvec = static_cast<int>((static_cast<int64_t>(V) * (dt == FEF_F32 ? 4 : 2)) / 16);
    int64_t parts = (4ll * sm_count) / rows;  // all CTAs resident at once where the rows are few
    const int64_t by_size = nvec / kDraftThreads;
    if (parts > by_size) parts = by_size;
    if (parts > kDraftMaxParts) parts = kDraftMaxParts;
    if (parts < 1) parts = 1;
    return static_cast<int>(parts);
}

static size_t draft_round256(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }

}  // namespace fef

extern "C" {

size_t fef_draft_sample_workspace_bytes(int B, int K, int V, fef_dtype dt) {
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V < 1) return 0;
    if (dt != FEF_F32 && dt != FEF_BF16) return 0;
    const size_t rows = static_cast<size_t>(B) * K;
    return fef::draft_round256(rows * sizeof(unsigned)) +
           fef::draft_round256(rows * fef::kDraftMaxParts * sizeof(fef::DraftPart));
}

}  // extern "C"

template <int DT, bool GREEDY>
static void launch_draft(const fef::DraftParams& P, unsigned grid, cudaStream_t stream) {
    if (P.target)
        fef::draft_kernel<DT, GREEDY, true><<<grid, fef::kDraftThreads, 0, stream>>>(P);
    else
        fef::draft_kernel<DT, GREEDY, false><<<grid, fef::kDraftThreads, 0, stream>>>(P);
}

static fef_status draft_impl(const void* draft_logits, const int32_t* row_len, int B, int K, int V, int64_t ld,
                             fef_dtype dt, float temperature, uint64_t seed, uint32_t step,
                             const uint32_t* device_round, int32_t* draft_tokens, double* log2_norm, void* workspace,
                             size_t workspace_bytes, int32_t* device_status, void* cuda_stream,
                             const void* target_logits = nullptr, double* target_log2_norm = nullptr) {
    using namespace fef;
    if (dt != FEF_F32 && dt != FEF_BF16) return FEF_ERR_DTYPE;
    if (!draft_logits || !draft_tokens) return FEF_ERR_INVALID_ARG;
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V < 1 || ld < V) return FEF_ERR_INVALID_ARG;
    if (!(temperature >= 0.0f) || isinf(temperature)) return FEF_ERR_INVALID_ARG;
    const int esize = dt == FEF_F32 ? 4 : 2;
    if (static_cast<int64_t>(V) * esize > (1ll << 30)) return FEF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(draft_logits) & 15) || ((ld * esize) & 15)) return FEF_ERR_ALIGNMENT;
    if (target_logits && (reinterpret_cast<uintptr_t>(target_logits) & 15)) return FEF_ERR_ALIGNMENT;
    if ((target_logits != nullptr) != (target_log2_norm != nullptr)) return FEF_ERR_INVALID_ARG;
    int dev = -1, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return FEF_ERR_CUDA;
    const size_t need = fef_draft_sample_workspace_bytes(B, K, V, dt);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need) return FEF_ERR_WORKSPACE;

    const bool greedy = temperature == 0.0f;
    DraftParams P;
    P.logits = static_cast<const char*>(draft_logits);
    P.target = static_cast<const char*>(target_logits);
    P.target_log2_norm = target_log2_norm;
    P.row_len = row_len;
    P.B = B;
    P.K = K;
    P.V = V;
    P.vec_elems = static_cast<int>((static_cast<int64_t>(V) * esize) / 16 * 16 / esize);
    P.parts = draft_parts(B, K, V, dt, sms);
    P.ld_bytes = ld * esize;
    const double c = 1.4426950408889634074 / (greedy ? 1.0 : static_cast<double>(temperature));
    float c_hi = static_cast<float>(c);
    if (dt == FEF_F32) {
        if (static_cast<double>(c_hi) >= c) c_hi = nextafterf(c_hi, 0.0f);
        P.c_lo = static_cast<float>(c - static_cast<double>(c_hi));
        if (!(P.c_lo > 0.f)) return FEF_ERR_INVALID_ARG;
    } else {
        P.c_lo = 0.f;
    }
    P.c_hi = c_hi;
    if (!(P.c_hi > 0.f) || isinf(P.c_hi)) return FEF_ERR_INVALID_ARG;
    P.seed = seed;
    P.keys = philox_round_keys(seed);
    P.step = step;
    P.round = device_round;
    P.tokens = draft_tokens;
    P.log2_norm = log2_norm;
    const size_t rows = static_cast<size_t>(B) * K;
    char* ws = static_cast<char*>(workspace);
    P.arrivals = reinterpret_cast<unsigned*>(ws);
    P.part_out = reinterpret_cast<DraftPart*>(ws + draft_round256(rows * sizeof(unsigned)));
    P.status = device_status;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (device_status && cudaMemsetAsync(device_status, 0, sizeof(int32_t), stream) != cudaSuccess) return FEF_ERR_CUDA;
    // the rows' arrival counters start at zero; nothing else in the scratch needs a defined value
    if (P.parts > 1 && cudaMemsetAsync(ws, 0, rows * sizeof(unsigned), stream) != cudaSuccess) return FEF_ERR_CUDA;
    const unsigned grid = static_cast<unsigned>(rows * P.parts);
    if (dt == FEF_F32) {
        if (greedy)
            launch_draft<FEF_F32, true>(P, grid, stream);
        else
            launch_draft<FEF_F32, false>(P, grid, stream);
    } else {
        if (greedy)
            launch_draft<FEF_BF16, true>(P, grid, stream);
        else
            launch_draft<FEF_BF16, false>(P, grid, stream);
    }
    return cudaGetLastError() == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

extern "C" {

fef_status fef_draft_sample(const void* draft_logits, const int32_t* row_len, int B, int K, int V, int64_t ld,
                            fef_dtype dt, float temperature, uint64_t seed, uint32_t step, int32_t* draft_tokens,
                            double* log2_norm, void* workspace, size_t workspace_bytes, int32_t* device_status,
                            void* cuda_stream) {
    return draft_impl(draft_logits, row_len, B, K, V, ld, dt, temperature, seed, step, nullptr, draft_tokens, log2_norm,
                      workspace, workspace_bytes, device_status, cuda_stream);
}

fef_status fef_draft_sample_at_round(const void* draft_logits, const int32_t* row_len, int B, int K, int V, int64_t ld,
                                     fef_dtype dt, float temperature, uint64_t seed, uint32_t step,
                                     const uint32_t* device_round, int32_t* draft_tokens, double* log2_norm,
                                     void* workspace, size_t workspace_bytes, int32_t* device_status,
                                     void* cuda_stream) {
    if (!device_round) return FEF_ERR_INVALID_ARG;
    return draft_impl(draft_logits, row_len, B, K, V, ld, dt, temperature, seed, step, device_round, draft_tokens,
                      log2_norm, workspace, workspace_bytes, device_status, cuda_stream);
}

fef_status fef_draft_sample_with_target(const void* draft_logits, const void* target_logits, const int32_t* row_len,
                                        int B, int K, int V, int64_t ld, fef_dtype dt, float temperature,
                                        uint64_t seed, uint32_t step, const uint32_t* device_round,
                                        int32_t* draft_tokens, double* draft_log2_norm, double* target_log2_norm,
                                        void* workspace, size_t workspace_bytes, int32_t* device_status,
                                        void* cuda_stream) {
    if (!target_logits || !target_log2_norm) return FEF_ERR_INVALID_ARG;
    return draft_impl(draft_logits, row_len, B, K, V, ld, dt, temperature, seed, step, device_round, draft_tokens,
                      draft_log2_norm, workspace, workspace_bytes, device_status, cuda_stream, target_logits,
                      target_log2_norm);
}

}  // extern "C"

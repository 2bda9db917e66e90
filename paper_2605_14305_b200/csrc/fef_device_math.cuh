// Device helpers shared by the verification kernels and the draft-sampling kernel (sm_100a):
// the per-thread running softmax sum, the Gumbel pieces, the best-two record.
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"

namespace fef {

__device__ __forceinline__ void report(int32_t* status, int code) {
    if (status) atomicMax(status, code);
}

// Running state of one thread for one row: sum of 2^(l*c - ref) and, in greedy
// mode, the largest logit with its lowest index.
struct RowState {
    float ref, sum, best;
    int index;
    __device__ __forceinline__ void reset() {
        ref = kNoReference;
        sum = 0.f;
        best = -INFINITY;
        index = 0x7FFFFFFF;
    }
};

template <int DT, bool GREEDY>
__device__ __forceinline__ void absorb_vector(const uint4& w, int first_index, float c_hi, float c_lo,
                                              RowState& st) {
    constexpr int N = Elem<DT>::kPerVec;
    float l[N], e[N];
    unpack<DT>(w, l);
#pragma unroll
    for (int i = 0; i < N; ++i) e[i] = exp2_scaled<DT>(l[i], c_hi, c_lo, st.ref);
    float vs;
    if constexpr (N == 8)
        vs = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
    else
        vs = (e[0] + e[1]) + (e[2] + e[3]);

    if (!(vs <= kRescaleAbove)) {
        // Rare: the reference is missing or far too low (or the data is bad).
        // Move the reference to this vector's maximum and redo the vector.
        float vmax = l[0];
        bool bad = (l[0] != l[0]);
#pragma unroll
        for (int i = 1; i < N; ++i) {
            vmax = fmaxf(vmax, l[i]);
            bad = bad || (l[i] != l[i]);
        }
        if (bad || vmax == INFINITY) {
            st.sum = __int_as_float(0x7FC00000);  // NaN marks the row as unusable
        } else {
            const float nref = fmaf(vmax, c_lo, vmax * c_hi);
            st.sum *= ex2_approx(st.ref - nref);
            st.ref = nref;
#pragma unroll
            for (int i = 0; i < N; ++i) e[i] = exp2_scaled<DT>(l[i], c_hi, c_lo, nref);
            if constexpr (N == 8)
                vs = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
            else
                vs = (e[0] + e[1]) + (e[2] + e[3]);
            st.sum += vs;
        }
    } else {
        st.sum += vs;
    }

    if constexpr (GREEDY) {
        float vmax = l[0];
#pragma unroll
        for (int i = 1; i < N; ++i) vmax = fmaxf(vmax, l[i]);
        if (vmax > st.best) {  // strict: an earlier (lower) index keeps a tie
            int at = N - 1;
#pragma unroll
            for (int i = N - 2; i >= 0; --i)
                if (l[i] == vmax) at = i;
            st.best = vmax;
            st.index = first_index + at;
        }
    }
}

// Reference exponent for a row that has none yet: c * (largest element of the thread's
// first vector), or "none" when that vector holds no finite number.
template <int DT>
__device__ __forceinline__ float first_reference(const uint4& w, float c_hi, float c_lo) {
    constexpr int N = Elem<DT>::kPerVec;
    float l[N];
    unpack<DT>(w, l);
    float vmax = l[0];
#pragma unroll
    for (int i = 1; i < N; ++i) vmax = fmaxf(vmax, l[i]);
    // (rounded to an integer: two partial sums of a row are then brought to a common reference by an exact
    // power of two, which the fold builds from the exponent instead of calling exp2)
    return (vmax > -INFINITY && vmax < INFINITY) ? rintf(fmaf(vmax, c_lo, vmax * c_hi)) : kNoReference;
}

// Monotone map between floats without NaN and signed integers (for integer warp reductions).
__device__ __forceinline__ int float_order(float f) {  // monotone map, floats without NaN -> int
    const int bits = __float_as_int(f);
    return bits >= 0 ? bits : (bits ^ 0x7FFFFFFF);
}
__device__ __forceinline__ float float_unorder(int k) {
    return __int_as_float(k >= 0 ? k : (k ^ 0x7FFFFFFF));
}
// For u = ((word >> 9) + 0.5) * 2^-23:  t = 1 - u (exact in binary32) and -ln(u), accurate
// also when u is close to 1.  Always -ln(u) > t.
__device__ __forceinline__ float one_minus_uniform(uint32_t word) {
    // k = word >> 9;  2^23 + (2^23 - 1 - k) assembled in the mantissa, then one exact multiply-add
    const float f = __uint_as_float(0x4B000000u | (~word >> 9));
    return fmaf(f, 1.0f / 8388608.0f, -(1.0f - 1.0f / 16777216.0f));
}
__device__ __forceinline__ float neg_log_uniform(float t) {
    const float series = t * fmaf(t, fmaf(t, fmaf(t, 0.25f, 1.0f / 3.0f), 0.5f), 1.0f);
    const float direct = -0.6931471805599453f * lg2_approx(1.0f - t);  // 1 - t = u exactly
    return t < 0.015625f ? series : direct;
}

struct Top2 {
    float w1, w2;
    int x1, x2;
    __device__ __forceinline__ void clear() {
        w1 = w2 = 0.f;
        x1 = x2 = 0x7FFFFFFF;
    }
    __device__ __forceinline__ void offer(float w, int x) {
        if (better(w, x, w1, x1)) {
            w2 = w1;
            x2 = x1;
            w1 = w;
            x1 = x;
        } else if (better(w, x, w2, x2)) {
            w2 = w;
            x2 = x;
        }
    }
    // best two of the whole warp, in every lane
    __device__ __forceinline__ void warp_merge() {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ow1 = __shfl_xor_sync(0xFFFFFFFFu, w1, o), ow2 = __shfl_xor_sync(0xFFFFFFFFu, w2, o);
            const int ox1 = __shfl_xor_sync(0xFFFFFFFFu, x1, o), ox2 = __shfl_xor_sync(0xFFFFFFFFu, x2, o);
            offer(ow1, ox1);
            offer(ow2, ox2);
        }
    }
};

__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// The three largest (weight, lowest id) a thread, warp or CTA has seen; empty slots hold weight 0.
struct Top3 {
    float w1, w2, w3;
    int x1, x2, x3;
    __device__ __forceinline__ void clear() {
        w1 = w2 = w3 = 0.f;
        x1 = x2 = x3 = 0x7FFFFFFF;
    }
    __device__ __forceinline__ void offer(float w, int x) {
        if (better(w, x, w1, x1)) {
            w3 = w2;
            x3 = x2;
            w2 = w1;
            x2 = x1;
            w1 = w;
            x1 = x;
        } else if (better(w, x, w2, x2)) {
            w3 = w2;
            x3 = x2;
            w2 = w;
            x2 = x;
        } else if (better(w, x, w3, x3)) {
            w3 = w;
            x3 = x;
        }
    }
    // Best three of the whole warp, in every lane: three rounds of "largest head over the lanes wins and
    // its lane moves on to its next entry" (weights are >= 0, so their bit patterns order like the values;
    // among equal weights the lowest id wins, as in offer()).
    __device__ __forceinline__ void warp_merge() {
        float rw[3];
        int rx[3];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const unsigned head = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(w1));
            const bool holder = __float_as_uint(w1) == head;
            const int id = __reduce_min_sync(0xFFFFFFFFu, holder ? x1 : 0x7FFFFFFF);
            rw[r] = __uint_as_float(head);
            rx[r] = id;
            if (holder && x1 == id) {
                w1 = w2;
                x1 = x2;
                w2 = w3;
                x2 = x3;
                w3 = 0.f;
                x3 = 0x7FFFFFFF;
            }
        }
        w1 = rw[0];
        x1 = rx[0];
        w2 = rw[1];
        x2 = rx[1];
        w3 = rw[2];
        x3 = rx[2];
    }
};

}  // namespace fef

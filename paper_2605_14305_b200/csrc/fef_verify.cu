// fef_spec_verify: the verification loop of the paper's Algorithm 2 for B windows at once.
//
// Three kernels, enqueued back to back on the caller's stream and chained with programmatic
// dependent launch:
//   begin_call_kernel  the claim counter, the windows' arrival counters and the caller's status
//                    word start at zero;
//   stream_kernel    reads every target and draft row exactly once (bulk-async copies into a
//                    shared-memory ring; persistent CTAs take runs of tiles, "claims", from a
//                    shared counter in row order) and leaves, per claim, the partial sum of
//                    2^(l_v * c - ref), c = log2(e) / T, from which pi(x) and rho(x) follow
//                    for any x  (the two softmax laws of Section 3.2);
//                    rows_kernel (many short rows) and small_rows_kernel (calls that stream little)
//                    take its place where the ring is a poor fit;
//   tail_kernel      grid (shares, windows): finishes the normalisers in double precision, draws
//                    u_i, applies u_i <= min{1, pi_i(x_i) / rho_i(x_i)}, finds the first rejection,
//                    writes accepted tokens and confidences c_i = pi_i(x_i); then, for windows that
//                    rejected, the Gumbel-max draw from [pi - rho]_+ over the rejected row (the
//                    residual law defined before Algorithm 2) and c = pi(Z).
// Greedy mode (temperature 0) ends with scan_kernel instead: arg-max compare, no random numbers.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"
#include "fef_device_math.cuh"
#include "fef_verify_params.cuh"
#include "fef_residual.cuh"

namespace fef {

// ============================================================ streaming ====
// One 16-byte vector, packed two-wide binary32 arithmetic (fma.rn.f32x2 / add.f32x2):
// adds 2^(l*c - ref) of its elements to two running pair-sums.  No overflow check here.
template <int DT>
__device__ __forceinline__ void add_vector_packed(const uint4& w, float2 ch, float2 cl, float2 nref,
                                                  float2& acc0, float2& acc1) {
    float2 l[4];
    if constexpr (DT == FEF_F32) {
        l[0] = make_float2(__uint_as_float(w.x), __uint_as_float(w.y));
        l[1] = make_float2(__uint_as_float(w.z), __uint_as_float(w.w));
    } else {
        l[0] = make_float2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u));
        l[1] = make_float2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
        l[2] = make_float2(__uint_as_float(w.z << 16), __uint_as_float(w.z & 0xFFFF0000u));
        l[3] = make_float2(__uint_as_float(w.w << 16), __uint_as_float(w.w & 0xFFFF0000u));
    }
#pragma unroll
    for (int k = 0; k < Elem<DT>::kPerVec / 2; ++k) {
        float2 x = __ffma2_rn(l[k], ch, nref);
        if constexpr (Elem<DT>::kSplitScale) x = __ffma2_rn(l[k], cl, x);
        const float2 e = make_float2(ex2_approx(x.x), ex2_approx(x.y));
        if (k & 1)
            acc1 = __fadd2_rn(acc1, e);
        else
            acc0 = __fadd2_rn(acc0, e);
    }
}

// A thread's share of one tile in sampling mode: the vectors with offset < len, one
// overflow check for the whole tile.  When the check fires (reference far too low or
// missing, or bad data) the tile is redone vector by vector through absorb_vector,
// which moves the reference.  Returns the thread's sum over the tile relative to st.ref, or
// NaN when the tile went the slow way.
template <int DT, bool FULL>
__device__ __forceinline__ float absorb_tile(const uint4 (&w)[kVecPerThread], const int (&at)[kVecPerThread], int len,
                                            float c_hi, float c_lo, RowState& st) {
    const float2 ch = make_float2(c_hi, c_hi);
    const float2 cl = make_float2(c_lo, c_lo);
    const float2 nref = make_float2(-st.ref, -st.ref);
    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j)
        if (FULL || at[j] < len) add_vector_packed<DT>(w[j], ch, cl, nref, acc0, acc1);
    const float2 acc = __fadd2_rn(acc0, acc1);
    const float ts = acc.x + acc.y;
    if (ts <= kRescaleAbove) {
        st.sum += ts;
        return ts;
    }
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j)
        if (FULL || at[j] < len) absorb_vector<DT, false>(w[j], 0, c_hi, c_lo, st);
    return __int_as_float(0x7FC00000);
}

// Butterfly over the warp: every lane ends with the combination of all 32 records
// (same tree in every lane, so the result does not depend on who asks).
// Greedy mode: largest logit of the thread's share and its lowest index.  The exact update below
// (unpack, compare, find the index) runs only for tiles that can hold a new maximum: a thread's
// tile sum of 2^(l c - ref), which the streaming pass computes anyway, is at least the largest
// of its terms, so a sum below 2^(floor c - ref) rules the whole tile out.  The floor is the
// warp's running maximum (refreshed once per tile); an element equal to it in a later tile has a
// higher index than its holder, so it need not be looked at.
template <int DT>
__device__ __forceinline__ void track_best(const uint4& w, int first_index, RowState& st) {
    constexpr int N = Elem<DT>::kPerVec;
    float l[N];
    unpack<DT>(w, l);
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

template <bool GREEDY>
__device__ __forceinline__ Partial warp_combine(float ref, float sum, float best, int index) {
    float M = ref;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, o));
    float s = sum * ex2_approx(ref - M);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if constexpr (GREEDY) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, index, o);
            if (better(ob, oi, best, index)) {
                best = ob;
                index = oi;
            }
        }
    }
    Partial p;
    p.ref = M;
    p.sum = s;
    p.best = best;
    p.index = index;
    return p;
}

// First kernel of a call: the claim counter, the windows' arrival counters (residual draw) and the
// caller's status word start at zero.  (One small kernel chained with programmatic dependent
// launch instead of memset nodes.)
constexpr int kBeginThreads = 128;
__global__ void __launch_bounds__(kBeginThreads) begin_call_kernel(Control* ctl, ResidualTask* tasks, int B, int32_t* status) {
    cudaGridDependencySynchronize();  // an earlier call on the stream may still be using them
    if (threadIdx.x == 0) {
        if (ctl) {
            ctl->next_claim = 0ull;
            ctl->aborted = 0;
        }
        if (status) *status = 0;
    }
    if (tasks)
        for (int b = threadIdx.x; b < B; b += kBeginThreads) tasks[b].arrivals = 0u;
}

enum : int { kFlagFirst = 1, kFlagLast = 2, kFlagExit = 4 };

// What a ring stage holds; written by the producer before the stage's barrier is armed.
struct __align__(16) StageDesc {
    int flags;      // kFlagFirst / kFlagLast tile of its claim; kFlagExit: no more stages
    int len;        // bytes in the stage (0: the claim has nothing to read)
    int offset;     // byte offset of the tile in its row
    unsigned slot;  // claim number (index of its partial)
};

// Shared memory behind the ring.
struct SharedControl {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    StageDesc desc[kStages];
    Partial slots[kSlotSets * kConsumerWarps];  // in-CTA combine buffers
    unsigned slot_count[kSlotSets];
    int abort_flag;
};
constexpr size_t kSmemBytes = static_cast<size_t>(kStages) * kTileBytes + sizeof(SharedControl);

template <int DT, bool GREEDY>
__global__ void __launch_bounds__(kStreamThreads, 1) stream_kernel(const __grid_constant__ VerifyParams P) {
    extern __shared__ __align__(128) unsigned char smem[];
    SharedControl& sc = *reinterpret_cast<SharedControl*>(smem + kStages * kTileBytes);
    uint64_t* full = sc.full;
    uint64_t* empty = sc.empty;
    volatile int* abort_flag = &sc.abort_flag;

    const Geometry& G = P.geo;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full + s, 1);
            mbar_init(empty + s, kConsumerWarps);
        }
        for (int s = 0; s < kSlotSets; ++s) sc.slot_count[s] = 0;
        sc.abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    cudaGridDependencySynchronize();  // begin_call_kernel has cleared the claim counter

    int issued = 0;  // stages put in flight (meaningful in the producer thread only)

    if (warp == kProducerWarp) {
        // ------------------------------------------------ producer (one thread)
        if (lane == 0) {
            bool ok = true;
            const uint64_t policy = l2_evict_first_policy();
            int next_stage = 0;
            uint32_t next_phase = 0;
            // the next free stage, or false after a bounded wait ran out
            auto acquire = [&](int& s) -> bool {
                s = next_stage;
                if (!mbar_wait_bounded(empty + s, next_phase ^ 1u, abort_flag, P.wait_limit_ns)) {
                    *abort_flag = 1;
                    P.ctl->aborted = 1;
                    report(P.status, FEF_ERR_TIMEOUT);
                    return false;
                }
                if (++next_stage == kStages) {
                    next_stage = 0;
                    next_phase ^= 1u;
                }
                return true;
            };

            // Claims are handed out in row order from a shared counter, so all CTAs stream one
            // compact, advancing region of memory and finish together.  Tickets are drawn two
            // ahead so that their round trip never holds up the ring.
            unsigned long long ticket = atomicAdd(&P.ctl->next_claim, 1ull);
            unsigned long long ticket_next = atomicAdd(&P.ctl->next_claim, 1ull);
            while (ok && ticket < static_cast<unsigned long long>(G.num_claims)) {
#ifdef FEF_TEST_HOOKS
                // Test build: this CTA's producer stops before the stage of the given number: nothing is
                // copied and nothing arrives for it, so the consumers' wait for that stage runs out.
                if (blockIdx.x == 0 && P.withhold_stage >= 0 && issued >= P.withhold_stage) {
                    ok = false;
                    break;
                }
#endif
                // 32-bit index arithmetic: this thread's instruction count per tile bounds how
                // fast the ring can be fed
                const unsigned claim = static_cast<unsigned>(ticket);
                ticket = ticket_next;
                ticket_next = atomicAdd(&P.ctl->next_claim, 1ull);
                const unsigned cpu = static_cast<unsigned>(G.claims_per_unit);
                const unsigned unit = cpu == 1u ? claim : claim / cpu;
                const unsigned ci = claim - unit * cpu;
                const unsigned row = G.units_per_row == 2 ? (unit >> 1) : unit;
                const bool is_draft = G.units_per_row == 2 && (unit & 1u);
                const unsigned b = row / static_cast<unsigned>(G.K);
                const int i = static_cast<int>(row - b * static_cast<unsigned>(G.K));
                const int n = P.row_len ? __ldg(P.row_len + b) : G.K;
                const char* base = (is_draft ? P.draft : P.target) + static_cast<int64_t>(row) * G.ld_bytes;
                const int t_begin = static_cast<int>(ci) * G.tiles_per_claim;
                const int t_end = min(t_begin + G.tiles_per_claim, G.tiles_per_unit);
                StageDesc d;
                d.slot = claim;
                if (i >= n || t_end <= t_begin) {
                    // nothing to read: an empty stage still produces the claim's (empty) partial
                    int s;
                    if (!(ok = acquire(s))) break;
                    d.flags = kFlagFirst | kFlagLast;
                    d.len = 0;
                    d.offset = 0;
                    sc.desc[s] = d;
                    mbar_arrive(full + s);
                    ++issued;
                } else {
                    int offset = t_begin * G.tile_bytes;
                    for (int t = t_begin; t < t_end; ++t, offset += G.tile_bytes) {
                        int s;
                        if (!(ok = acquire(s))) break;
                        const int len = min(G.tile_bytes, G.vec_bytes - offset);
                        d.flags = (t == t_begin ? kFlagFirst : 0) | (t == t_end - 1 ? kFlagLast : 0);
                        d.len = len;
                        d.offset = offset;
                        sc.desc[s] = d;
                        mbar_arrive_expect_tx(full + s, static_cast<uint32_t>(len));
                        bulk_copy_g2s(smem + s * kTileBytes, base + offset, static_cast<uint32_t>(len), full + s, policy);
                        ++issued;
                    }
                }
            }
            if (ok) {
                int s;
                if (acquire(s)) {
                    StageDesc d = {};
                    d.flags = kFlagExit;
                    sc.desc[s] = d;
                    mbar_arrive(full + s);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        RowState st;
        st.reset();
        int s = 0;
        uint32_t phase = 0;
        int flushes = 0;  // combines done (same sequence in every consumer warp)
        while (true) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(full + s, phase, abort_flag, P.wait_limit_ns))) {
                *abort_flag = 1;
                if (lane == 0) P.ctl->aborted = 1;
                report(P.status, FEF_ERR_TIMEOUT);
                break;
            }
            const StageDesc d = sc.desc[s];
            if (d.flags & kFlagExit) break;
            const unsigned char* stage = smem + s * kTileBytes;

            if (d.flags & kFlagFirst) st.reset();
            const int s_cur = s;
            if (++s == kStages) {
                s = 0;
                phase ^= 1u;
            }
            // a tile is taken in chunks of kVecPerThread vectors per thread: the wait, the descriptor
            // and the release are paid once per tile, the registers hold one chunk
#pragma unroll
            for (int h = 0; h < kHalves; ++h) {
                const int hbase = h * kChunkBytes;
                uint4 w[kVecPerThread];
                int at[kVecPerThread];
#pragma unroll
                for (int j = 0; j < kVecPerThread; ++j) {
                    at[j] = hbase + ((j * kConsumerWarps + warp) * 32 + lane) * 16;
                    if (at[j] < d.len) w[j] = *reinterpret_cast<const uint4*>(stage + at[j]);
                }
                if (h == kHalves - 1) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty + s_cur);  // the stage may be refilled
                }
                if (d.len > hbase) {
                    if (st.ref == kNoReference && at[0] < d.len) st.ref = first_reference<DT>(w[0], P.c_hi, P.c_lo);
                    float tile_sum;
                    if (d.len >= hbase + kChunkBytes)  // branch-free: the four vectors interleave
                        tile_sum = absorb_tile<DT, true>(w, at, d.len, P.c_hi, P.c_lo, st);
                    else
                        tile_sum = absorb_tile<DT, false>(w, at, d.len, P.c_hi, P.c_lo, st);
                    if constexpr (GREEDY) {
                        const float floor_f = float_unorder(__reduce_max_sync(0xFFFFFFFFu, float_order(st.best)));
                        // 0.999: the sum and the bound carry a few units of 1e-7 of rounding each
                        const bool candidate = !(tile_sum < 0.999f * exp2_scaled<DT>(floor_f, P.c_hi, P.c_lo, st.ref));
                        if (__any_sync(0xFFFFFFFFu, candidate)) {  // the vote keeps this out of the straight-line code
                            if (candidate) {
#pragma unroll
                                for (int j = 0; j < kVecPerThread; ++j)
                                    if (at[j] < d.len)
                                        track_best<DT>(w[j], (d.offset + at[j]) / Elem<DT>::kBytes, st);
                            }
                        }
                    }
                }
            }
            if (d.flags & kFlagLast) {
                // claim finished: warp result -> combine slot; the last warp to arrive folds the 16
                // records and stores the claim's partial (read by the next kernel)
                const Partial mine = warp_combine<GREEDY>(st.ref, st.sum, st.best, st.index);
                const int set = flushes % kSlotSets;
                ++flushes;
                unsigned before = 0;
                if (lane == 0) {
                    sc.slots[set * kConsumerWarps + warp] = mine;
                    __threadfence_block();
                    before = atomicAdd(sc.slot_count + set, 1u);
                }
                before = __shfl_sync(0xFFFFFFFFu, before, 0);
                if (before == kConsumerWarps - 1) {
                    __threadfence_block();
                    Partial rec;
                    rec.ref = kNoReference;
                    rec.sum = 0.f;
                    rec.best = -INFINITY;
                    rec.index = 0x7FFFFFFF;
                    if (lane < kConsumerWarps) rec = sc.slots[set * kConsumerWarps + lane];
                    const Partial all = warp_combine<GREEDY>(rec.ref, rec.sum, rec.best, rec.index);
                    if (lane == 0) {
                        sc.slot_count[set] = 0;
                        P.partials[d.slot] = all;
                    }
                }
            }
        }
    }

    __syncthreads();
    // After an abort copies may still be in flight into this CTA's shared memory:
    // give each a bounded chance to land before the CTA retires.
    if (*abort_flag && warp == kProducerWarp && lane == 0) {
        const int first = issued > kStages ? issued - kStages : 0;
        for (int k = first; k < issued; ++k) {
            const int s = k % kStages;
            const uint32_t phase = (k / kStages) & 1;
            volatile int never = 0;
            mbar_wait_bounded(full + s, phase, &never, P.wait_limit_ns);
        }
    }
}

// ========================================================= short rows ====
// The same sums for rows that fit one tile when there are many of them (small vocabularies,
// slices of a sharded vocabulary): one warp per row and tensor, four 16-byte loads per lane in
// flight, one warp reduction per row, no shared memory.  Leaves one partial per row like the ring.
constexpr int kRowsWarps = 8;        // rows a CTA works on at a time
constexpr int kRowsCtasPerSm = 3;  // (four would cap the kernel at 64 registers: it spilled up to 412 bytes there; two leave no
                                   // spill at all but run vocabulary slices 3-4 % slower than three with their few bytes)

template <int DT, bool GREEDY>
__global__ void __launch_bounds__(kRowsWarps * 32, kRowsCtasPerSm) rows_kernel(const __grid_constant__ VerifyParams P) {
    const Geometry& G = P.geo;
    cudaGridDependencySynchronize();  // an earlier call on the stream may still be reading the partials
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kRowsWarps;
    for (int64_t unit = static_cast<int64_t>(blockIdx.x) * kRowsWarps + warp; unit < G.num_units; unit += stride) {
        const int64_t row = G.units_per_row == 2 ? (unit >> 1) : unit;
        const bool is_draft = G.units_per_row == 2 && (unit & 1);
        const int b = static_cast<int>(row / G.K), i = static_cast<int>(row - static_cast<int64_t>(b) * G.K);
        const int n = P.row_len ? __ldg(P.row_len + b) : G.K;
        RowState st;
        st.reset();
        if (i < n) {
            const char* base = (is_draft ? P.draft : P.target) + row * G.ld_bytes;
            const int len = G.vec_bytes;
            // two batches of four vectors per lane are in flight: the second is issued before the first
            // is added up
            constexpr int kBatchBytes = 32 * 16 * kVecPerThread;
            // (the loop bounds are the same in every lane: the warp votes of greedy mode need the whole warp)
            for (int off = 0; off < len; off += 2 * kBatchBytes) {
                uint4 w[2][kVecPerThread];
                int at[2][kVecPerThread];
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int j = 0; j < kVecPerThread; ++j) {
                        at[h][j] = off + h * kBatchBytes + j * 32 * 16 + lane * 16;
                        if (at[h][j] < len) w[h][j] = ld_global_nc_v4(base + at[h][j]);
                    }
                if (st.ref == kNoReference && at[0][0] < len) st.ref = first_reference<DT>(w[0][0], P.c_hi, P.c_lo);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (off + h * kBatchBytes >= len) break;  // uniform over the warp
                    float tile_sum;
                    if (at[h][kVecPerThread - 1] < len)
                        tile_sum = absorb_tile<DT, true>(w[h], at[h], len, P.c_hi, P.c_lo, st);
                    else
                        tile_sum = absorb_tile<DT, false>(w[h], at[h], len, P.c_hi, P.c_lo, st);
                    if constexpr (GREEDY) {
                        const float floor_f = float_unorder(__reduce_max_sync(0xFFFFFFFFu, float_order(st.best)));
                        // 0.999: the sum and the bound carry a few units of 1e-7 of rounding each
                        const bool candidate = !(tile_sum < 0.999f * exp2_scaled<DT>(floor_f, P.c_hi, P.c_lo, st.ref));
                        if (__any_sync(0xFFFFFFFFu, candidate)) {
                            if (candidate) {
#pragma unroll
                                for (int j = 0; j < kVecPerThread; ++j)
                                    if (at[h][j] < len) track_best<DT>(w[h][j], at[h][j] / Elem<DT>::kBytes, st);
                            }
                        }
                    }
                }
            }
        }
        const Partial all = warp_combine<GREEDY>(st.ref, st.sum, st.best, st.index);
        if (lane == 0) P.partials[unit] = all;
    }
}

// ================================================================= scan ====
struct RowNorm {
    double M;     // reference exponent (log2 domain)
    double S;     // sum_v 2^(l_v c - M)
    float best;   // greedy: largest logit
    int index;    // greedy: its lowest index
    bool bad;
    bool data_bad; // a NaN or +inf was seen (bad also covers rows without any finite logit)
};

// 2^d for the difference d <= 0 of two reference exponents.  The streaming kernels round their references
// to integers, so d is an integer unless a sum had to be re-referenced: then the power is assembled from its
// exponent (exact) instead of going through exp2.
__device__ __forceinline__ double pow2_of_difference(double d) {
    const int n = static_cast<int>(d);
    if (static_cast<double>(n) == d && n > -1000 && n <= 0) return __hiloint2double((1023 + n) << 20, 0);
    return exp2(d);
}

// Fold the claims' partials of unit u (and the row's tail elements, which the streaming
// kernel does not touch) into the row's normaliser.  One thread.
template <int DT, bool GREEDY>
__device__ __forceinline__ RowNorm fold_unit(int64_t u, const char* row, double c, const VerifyParams& P) {
    const Geometry& G = P.geo;
    const int nrec = G.claims_per_unit;
    const Partial* rec = P.partials + u * G.claims_per_unit;
    double m = -INFINITY, sacc = 0.0;
    bool bad = false;
    float best = -INFINITY;
    int index = 0x7FFFFFFF;
    for (int r = 0; r < nrec; ++r) {
        const Partial p = rec[r];
        if (!(p.sum >= 0.f) || p.sum == INFINITY) bad = true;
        if (p.sum > 0.f) {
            const double pm = p.ref, ps = p.sum;
            if (pm > m) {  // (the first record, and any record equal to the running reference, needs no scaling)
                sacc = m > -INFINITY ? sacc * pow2_of_difference(m - pm) + ps : ps;
                m = pm;
            } else {
                sacc += pm == m ? ps : ps * pow2_of_difference(pm - m);
            }
        }
        if (GREEDY && better(p.best, p.index, best, index)) {
            best = p.best;
            index = p.index;
        }
    }
    for (int x = G.vec_elems; x < G.V; ++x) {
        const float l = load_logit<DT>(row, x);
        if (l != l || l == INFINITY) {
            bad = true;
        } else if (l > -INFINITY) {
            const double pm = static_cast<double>(l) * c;
            if (pm > m) {
                sacc = sacc * exp2(m - pm) + 1.0;
                m = pm;
            } else {
                sacc += exp2(pm - m);
            }
        }
        if (GREEDY && better(l, x, best, index)) {
            best = l;
            index = x;
        }
    }
    RowNorm out;
    out.M = m;
    out.S = sacc;
    out.best = best;
    out.index = index;
    out.bad = bad || !(sacc > 0.0) || !(sacc < INFINITY);
    out.data_bad = bad || !(sacc < INFINITY) || sacc != sacc;
    return out;
}

constexpr int kScanWarps = 4;  // windows per CTA of the scan kernel

// Greedy mode (temperature 0), after the streaming kernel: a draft is accepted iff it is the arg-max
// of the target logits; the first rejection is replaced by that arg-max; confidences are the
// T = 1 softmax probabilities.  One warp per window, lane l does positions l and l + 32.
template <int DT>
__global__ void __launch_bounds__(kScanWarps * 32) scan_kernel(const __grid_constant__ VerifyParams P) {
    const Geometry& G = P.geo;
    constexpr int kRounds = FEF_MAX_K / 32;
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * kScanWarps + (threadIdx.x >> 5);
    if (b >= G.B) return;
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), G.K) : G.K;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);

    // what does not depend on the streaming kernel is fetched before waiting for it
    int tok[kRounds];
    double lpx[kRounds];
#pragma unroll
    for (int r = 0; r < kRounds; ++r) {
        const int i = r * 32 + lane;
        tok[r] = -1;
        lpx[r] = 0.0;
        if (r * 32 < G.K && i < n) {
            const int64_t row = static_cast<int64_t>(b) * G.K + i;
            const int x = __ldg(P.draft_tokens + row);
            tok[r] = x;
            if (x >= 0 && x < G.V) lpx[r] = load_logit<DT>(P.target + row * G.ld_bytes, x);
        }
    }
    cudaGridDependencySynchronize();  // the streaming kernel's partials must be complete and visible
    const bool aborted = P.ctl->aborted != 0;  // a wait in the streaming kernel ran out: no window is decided

    int alt[kRounds];
    float cf[kRounds], cf_alt[kRounds];
    unsigned rejected[kRounds];
    int err = 0;
#pragma unroll
    for (int r = 0; r < kRounds; ++r) {
        const int i = r * 32 + lane;
        alt[r] = -1;
        cf[r] = cf_alt[r] = -1.f;
        bool accept = true;
        if (r * 32 < G.K && i < n) {
            const int64_t row = static_cast<int64_t>(b) * G.K + i;
            const int x = tok[r];
            const RowNorm np = fold_unit<DT, true>(row * G.units_per_row, P.target + row * G.ld_bytes, c, P);
            if (x < 0 || x >= G.V) {
                err = max(err, static_cast<int>(FEF_ERR_TOKEN_RANGE));
            } else if (np.bad) {
                err = max(err, static_cast<int>(FEF_ERR_NONFINITE));
            } else {
                const double kp = np.M + log2(np.S);
                cf[r] = static_cast<float>(exp2(lpx[r] * c - kp));
                accept = (x == np.index);
                alt[r] = np.index;
                cf_alt[r] = static_cast<float>(exp2(static_cast<double>(np.best) * c - kp));
            }
        }
        rejected[r] = __ballot_sync(0xFFFFFFFFu, !accept);
    }
    err = __reduce_max_sync(0xFFFFFFFFu, err);
    if (aborted) err = FEF_ERR_TIMEOUT;

    int a = n;
#pragma unroll
    for (int r = kRounds - 1; r >= 0; --r)
        if (rejected[r]) a = r * 32 + __ffs(rejected[r]) - 1;

#pragma unroll
    for (int r = 0; r < kRounds; ++r) {
        const int i = r * 32 + lane;
        if (i < G.K) {
            const int64_t row = static_cast<int64_t>(b) * G.K + i;
            int t = -1;
            float f = -1.f;
            if (!err) {
                if (i < a) {
                    t = tok[r];
                    f = cf[r];
                } else if (i == a && a < n) {
                    t = alt[r];
                    f = cf_alt[r];
                }
            }
            P.tokens[row] = t;
            P.conf[row] = f;
        }
    }
    if (lane == 0) {
        P.accept_len[b] = err ? -1 : a;
        if (err) report(P.status, err);
    }
}

// The same as fold_unit, done by a whole warp: the lanes share the unit's partials.
template <int DT, bool GREEDY>
__device__ RowNorm fold_unit_warp(int64_t u, const char* row, double c, const VerifyParams& P, int lane) {
    const Geometry& G = P.geo;
    const int nrec = G.claims_per_unit;
    const Partial* rec = P.partials + u * G.claims_per_unit;
    const int ntail = G.V - G.vec_elems;

    // each lane folds its records into a running (m, s) pair, then the warp combines
    double m = -INFINITY, sacc = 0.0;
    int bad = 0;
    float best = -INFINITY;
    int index = 0x7FFFFFFF;
    for (int r = lane; r < nrec; r += 32) {
        const Partial p = rec[r];
        if (!(p.sum >= 0.f) || p.sum == INFINITY) bad = 1;
        if (p.sum > 0.f) {
            const double pm = p.ref, ps = p.sum;
            if (pm > m) {  // (the first record, and any record equal to the running reference, needs no scaling)
                sacc = m > -INFINITY ? sacc * pow2_of_difference(m - pm) + ps : ps;
                m = pm;
            } else {
                sacc += pm == m ? ps : ps * pow2_of_difference(pm - m);
            }
        }
        if (GREEDY && better(p.best, p.index, best, index)) {
            best = p.best;
            index = p.index;
        }
    }
    for (int j = lane; j < ntail; j += 32) {
        const float l = load_logit<DT>(row, G.vec_elems + j);
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
        }
        if (GREEDY && better(l, G.vec_elems + j, best, index)) {
            best = l;
            index = G.vec_elems + j;
        }
    }
    const double M = warp_max(m);
    bad = __any_sync(0xFFFFFFFFu, bad);
    if (GREEDY) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, o);
            const int oi = __shfl_xor_sync(0xFFFFFFFFu, index, o);
            if (better(ob, oi, best, index)) {
                best = ob;
                index = oi;
            }
        }
    }
    const double S = warp_sum(m > -INFINITY ? sacc * pow2_of_difference(m - M) : 0.0);
    RowNorm out;
    out.M = M;
    out.S = S;
    out.best = best;
    out.index = index;
    out.bad = bad || !(S > 0.0) || !(S < INFINITY);
    out.data_bad = bad || !(S < INFINITY) || S != S;
    return out;
}

constexpr int kScanMaxWarps = 32;

// The same greedy step with one CTA per window and one warp per position, for calls whose rows are
// cut into many claims (few rows in all): the fold of a row's partials is then shared by 32 lanes.
template <int DT>
__global__ void __launch_bounds__(kScanMaxWarps * 32) scan_rows_kernel(const __grid_constant__ VerifyParams P) {
    const Geometry& G = P.geo;
    const int num_warps = blockDim.x >> 5;
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), G.K) : G.K;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);

    // what does not depend on the streaming kernel is fetched before waiting for it: the draft
    // tokens of this warp's positions and the logits at them (a warp has at most kRows positions)
    constexpr int kRows = (FEF_MAX_K + kScanMaxWarps - 1) / kScanMaxWarps;
    int pre_x[kRows];
    double pre_lp[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const int i = warp + r * num_warps;
        pre_x[r] = -1;
        pre_lp[r] = 0.0;
        if (lane == 0 && i < n) {
            const int64_t row = static_cast<int64_t>(b) * G.K + i;
            const int x = __ldg(P.draft_tokens + row);
            pre_x[r] = x;
            if (x >= 0 && x < G.V) pre_lp[r] = load_logit<DT>(P.target + row * G.ld_bytes, x);
        }
    }
    cudaGridDependencySynchronize();  // the streaming kernel's partials must be complete and visible

    __shared__ float s_conf[FEF_MAX_K], s_conf_alt[FEF_MAX_K];
    __shared__ int s_accept[FEF_MAX_K], s_err[FEF_MAX_K], s_alt[FEF_MAX_K];

#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const int i = warp + r * num_warps;
        if (i >= n) break;  // uniform over the warp
        const int64_t row = static_cast<int64_t>(b) * G.K + i;
        const RowNorm np = fold_unit_warp<DT, true>(row * G.units_per_row, P.target + row * G.ld_bytes, c, P, lane);
        if (lane == 0) {
            const int x = pre_x[r];
            int err = 0, accept = 0, alt = -1;
            float conf = -1.f, conf_alt = -1.f;
            if (x < 0 || x >= G.V) {
                err = FEF_ERR_TOKEN_RANGE;
            } else if (np.bad) {
                err = FEF_ERR_NONFINITE;
            } else {
                const double kp = np.M + log2(np.S);
                conf = static_cast<float>(exp2(pre_lp[r] * c - kp));
                accept = (x == np.index);
                alt = np.index;
                conf_alt = static_cast<float>(exp2(static_cast<double>(np.best) * c - kp));
            }
            s_err[i] = err;
            s_accept[i] = accept;
            s_conf[i] = conf;
            s_conf_alt[i] = conf_alt;
            s_alt[i] = alt;
        }
    }
    __syncthreads();

    int err = 0, a = n;
    for (int i = 0; i < n; ++i) err = max(err, s_err[i]);
    if (P.ctl->aborted) err = FEF_ERR_TIMEOUT;  // a wait in the streaming kernel ran out: no window is decided
    for (int i = n - 1; i >= 0; --i)
        if (!s_accept[i]) a = i;

    for (int i = threadIdx.x; i < G.K; i += blockDim.x) {
        const int64_t row = static_cast<int64_t>(b) * G.K + i;
        int tok = -1;
        float cf = -1.f;
        if (!err) {
            if (i < a) {
                tok = __ldg(P.draft_tokens + row);
                cf = s_conf[i];
            } else if (i == a && a < n) {
                tok = s_alt[i];
                cf = s_conf_alt[i];
            }
        }
        P.tokens[row] = tok;
        P.conf[row] = cf;
    }
    if (threadIdx.x == 0) {
        P.accept_len[b] = err ? -1 : a;
        if (err) report(P.status, err);
    }
}


// ============================================================= residual ====
// (the draw itself: fef_residual.cuh)

// Vocabulary-parallel mode: the residual draw over this rank's slice for the windows whose task
// (written by vp_accept_kernel) names a rejected position.
template <int DT>
__global__ void __launch_bounds__(kResidualThreads, kResidualCtasPerSm) residual_kernel(const __grid_constant__ VerifyParams P) {
    __shared__ ResidualShared sh;
    cudaGridDependencySynchronize();
    const int b = blockIdx.y;
    const ResidualTask task = P.tasks[b];
    if (task.pos < 0) return;  // uniform over the CTA
    if (threadIdx.x == 0) sh.floor_bits = sh.best3[0] = sh.best3[1] = sh.best3[2] = 0u;
    __syncthreads();
    const int64_t row = static_cast<int64_t>(b) * P.geo.K + task.pos;
    residual_draw<DT, true, false>(P, b, task.pos, task.kp, task.kq, P.target + row * P.geo.ld_bytes,
                            P.draft + row * P.geo.ld_bytes, row, blockIdx.x, gridDim.x, sh);
}

// ================================================================= tail ====
// Sampling mode, everything after the streaming kernel in one launch (Algorithm 2, "for m = 1..b"
// from the acceptance test on): grid (parts, B).  Every CTA of window b repeats the window's
// acceptance tests from the partials (a few hundred operations per position, the same in every
// CTA, so all agree on the first rejection without talking to each other); part 0 writes the accepted
// tokens and confidences; then the CTAs share the residual draw of the rejected row.
struct TailShared {
    double kp[FEF_MAX_K], kq[FEF_MAX_K];
    float conf[FEF_MAX_K];
    int tok[FEF_MAX_K];
    unsigned rejected[FEF_MAX_K / 32];
    int err;
};

// One position's acceptance test from its folded normalisers.  Returns 0 or a data error.
__device__ __forceinline__ int accept_test(const VerifyParams& P, int b, int i, int x, double lpx, double lqx,
                                           const RowNorm& np, const RowNorm& nq, double c, TailShared& ts) {
    const Geometry& G = P.geo;
    if (x < 0 || x >= G.V) return FEF_ERR_TOKEN_RANGE;
    if (np.bad || nq.bad) return FEF_ERR_NONFINITE;
    const double kp = np.M + log2(np.S);
    const double kq = nq.M + log2(nq.S);
    const double l2pi = lpx * c - kp;  // log2 pi(x)
    bool accept;
    if (lqx == -INFINITY) {
        accept = lpx > -INFINITY;  // rho(x) = 0: accept iff pi(x) > 0
    } else {
        const double ratio = exp2(l2pi - (lqx * c - kq));
        const uint4 rnd = philox4x32_10(
            make_uint4(kStreamAccept << 30, static_cast<uint32_t>(b), static_cast<uint32_t>(i), step_of(P)),
            make_uint2(static_cast<uint32_t>(P.seed), static_cast<uint32_t>(P.seed >> 32)));
        accept = static_cast<double>(uniform_from_word(rnd.x)) <= fmin(1.0, ratio);
    }
    ts.kp[i] = kp;
    ts.kq[i] = kq;
    ts.conf[i] = static_cast<float>(exp2(l2pi));
    ts.tok[i] = x;
    if (!accept) atomicOr(&ts.rejected[i >> 5], 1u << (i & 31));
    return 0;
}

// What the acceptance tests need besides the normalisers, fetched before those are waited for: the
// draft token of "my" position and the two logits at it.  Thread form: position threadIdx.x.  Warp
// form (wide): lane j of warp w holds position w + j * kResidualWarps.
template <int DT>
__device__ __forceinline__ void fetch_my_position(const VerifyParams& P, int b, int n, bool wide, int& my, int& x,
                                                  double& lpx, double& lqx) {
    const Geometry& G = P.geo;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    my = wide ? (lane < FEF_MAX_K / kResidualWarps ? warp + lane * kResidualWarps : FEF_MAX_K)
              : static_cast<int>(threadIdx.x);
    x = -1;
    lpx = 0.0;
    lqx = 0.0;
    if (my < n) {
        const int64_t row = static_cast<int64_t>(b) * G.K + my;
        x = __ldg(P.draft_tokens + row);
        if (x >= 0 && x < G.V) {
            lpx = load_logit<DT>(P.target + row * G.ld_bytes, x);
            lqx = load_logit<DT>(P.draft + row * G.ld_bytes, x);
        }
    }
}

// The acceptance tests of window b from the partials (whole CTA; `ts` cleared and a barrier passed
// before).  Returns the first rejected position (n when every draft was accepted); ts.err holds a
// data error, if any.
template <int DT>
__device__ __forceinline__ int window_accept(const VerifyParams& P, int b, int n, bool wide, int my, int x, double lpx,
                                             double lqx, double c, TailShared& ts) {
    const Geometry& G = P.geo;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!wide) {
        if (my < n) {
            const int64_t row = static_cast<int64_t>(b) * G.K + my;
            if (G.claims_per_unit > 1) {
                // several partials per row, read one after the other below: have them all on their way to L1 first
                const Partial* recs = P.partials + row * G.units_per_row * G.claims_per_unit;
                for (int r = 0; r < G.units_per_row * G.claims_per_unit; r += 2)
                    asm volatile("prefetch.global.L1 [%0];" ::"l"(recs + r));
            }
            RowNorm np;
            if (P.target_norm) {  // both laws' normalisers came with the drafts: nothing was streamed
                np.M = P.target_norm[row];
                np.S = 1.0;
                np.bad = !(fabs(np.M) < INFINITY);
            } else {
                np = fold_unit<DT, false>(row * G.units_per_row, P.target + row * G.ld_bytes, c, P);
            }
            RowNorm nq;
            if (P.draft_norm) {  // rho(x) = 2^(l_x c - norm): the normaliser came with the drafts
                nq.M = P.draft_norm[row];
                nq.S = 1.0;
                nq.bad = !(fabs(nq.M) < INFINITY);
            } else {
                nq = fold_unit<DT, false>(2 * row + 1, P.draft + row * G.ld_bytes, c, P);
            }
            const int e = accept_test(P, b, my, x, lpx, lqx, np, nq, c, ts);
            if (e) atomicMax(&ts.err, e);
        }
    } else {
        for (int j = 0; j < FEF_MAX_K / kResidualWarps; ++j) {
            const int i = warp + j * kResidualWarps;
            if (i >= n) break;  // uniform over the warp
            const int64_t row = static_cast<int64_t>(b) * G.K + i;
            RowNorm np;
            if (P.target_norm) {
                np.M = P.target_norm[row];
                np.S = 1.0;
                np.bad = !(fabs(np.M) < INFINITY);
            } else {
                np = fold_unit_warp<DT, false>(row * G.units_per_row, P.target + row * G.ld_bytes, c, P, lane);
            }
            RowNorm nq;
            if (P.draft_norm) {
                nq.M = P.draft_norm[row];
                nq.S = 1.0;
                nq.bad = !(fabs(nq.M) < INFINITY);
            } else {
                nq = fold_unit_warp<DT, false>(2 * row + 1, P.draft + row * G.ld_bytes, c, P, lane);
            }
            const int xi = __shfl_sync(0xFFFFFFFFu, x, j);
            const double lpi = __shfl_sync(0xFFFFFFFFu, lpx, j), lqi = __shfl_sync(0xFFFFFFFFu, lqx, j);
            if (lane == 0) {
                const int e = accept_test(P, b, i, xi, lpi, lqi, np, nq, c, ts);
                if (e) atomicMax(&ts.err, e);
            }
        }
    }
    __syncthreads();
    int a = n;
    if (ts.rejected[0])
        a = __ffs(ts.rejected[0]) - 1;
    else if (ts.rejected[1])
        a = 32 + __ffs(ts.rejected[1]) - 1;
    return a;
}

// Window b's accepted tokens, confidences and length (one CTA of the window calls this).
__device__ __forceinline__ void write_window(const VerifyParams& P, int b, int a, int err, const TailShared& ts) {
    const Geometry& G = P.geo;
    for (int i = threadIdx.x; i < G.K; i += kResidualThreads) {
        const int64_t row = static_cast<int64_t>(b) * G.K + i;
        const bool keep = !err && i < a;
        P.tokens[row] = keep ? ts.tok[i] : -1;
        P.conf[row] = keep ? ts.conf[i] : -1.f;
    }
    if (threadIdx.x == 0) {
        P.accept_len[b] = err ? -1 : a;
        if (err) report(P.status, err);
    }
}
// A window that stays undecided (a wait ran out).
__device__ __forceinline__ void write_window_undecided(const VerifyParams& P, int b) {
    const Geometry& G = P.geo;
    for (int i = threadIdx.x; i < G.K; i += kResidualThreads) {
        P.tokens[static_cast<int64_t>(b) * G.K + i] = -1;
        P.conf[static_cast<int64_t>(b) * G.K + i] = -1.f;
    }
    if (threadIdx.x == 0) P.accept_len[b] = -1;
}

template <int DT, bool CLUSTER>
__global__ void __launch_bounds__(kResidualThreads, kResidualCtasPerSm) tail_kernel(const __grid_constant__ VerifyParams P) {
    const Geometry& G = P.geo;
    __shared__ TailShared ts;
    __shared__ ResidualShared sh;
    const int b = blockIdx.y, part = blockIdx.x;
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), G.K) : G.K;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);
    // very many partials per row: a warp per position shares the fold; otherwise a thread per position
    // (with eight warps and up to 64 positions, the serial fold of a few dozen partials is still faster)
    const bool wide = G.claims_per_unit > 32;

    int my, x;
    double lpx, lqx;
    fetch_my_position<DT>(P, b, n, wide, my, x, lpx, lqx);
    if (threadIdx.x == 0) {
        ts.rejected[0] = ts.rejected[1] = 0u;
        ts.err = 0;
        sh.floor_bits = sh.best3[0] = sh.best3[1] = sh.best3[2] = 0u;
    }
    __syncthreads();
    cudaGridDependencySynchronize();  // the streaming kernel's partials must be complete and visible

    if (P.ctl->aborted) {  // a wait in the streaming kernel ran out (status FEF_ERR_TIMEOUT): no window is decided
        if (part == 0) write_window_undecided(P, b);
        return;
    }

    const int a = window_accept<DT>(P, b, n, wide, my, x, lpx, lqx, c, ts);
    const int err = ts.err;
    if (part == 0) write_window(P, b, a, err, ts);
    if (err || a >= n) return;  // uniform over the CTA (and over the window's CTAs)
    const int64_t row = static_cast<int64_t>(b) * G.K + a;
    residual_draw<DT, false, CLUSTER>(P, b, a, ts.kp[a], ts.kq[a], P.target + row * G.ld_bytes,
                                                                    P.draft + row * G.ld_bytes, row, part,
                                                                    static_cast<int>(gridDim.x), sh);
}

// ============================================================ few rows ====
// Calls that stream little (sampling mode) replace the streaming kernel by one built for latency instead of
// bandwidth: grid (shares, windows), all CTAs resident; groups of warps (1, 2, 4 warps, or the 8 of one or
// several whole CTAs) each add up one row of the window, every lane with all its 16-byte loads of the row in
// flight at once.  The CTAs that share a row form a thread-block cluster and meet in the shared memory of
// its first CTA, so every row leaves one partial, as the acceptance tests of tail_kernel (which follows as
// usual) like it best.
constexpr int kSmallDepth = 4;  // batches of kVecPerThread vectors a lane has in flight
constexpr int64_t kSmallMaxBytes = 48ll << 20;  // calls that stream at most this much take this path
constexpr int kMaxSmallCtas = 1024;             // ... with at most this many CTAs in this kernel
constexpr int kSmallMaxCtasPerRow = 8;          // ... of which at most this many (one cluster) share a row

template <int DT, bool CLUSTER>
__global__ void __launch_bounds__(kResidualThreads, kResidualCtasPerSm) small_rows_kernel(const __grid_constant__ VerifyParams P) {
    const Geometry& G = P.geo;
    __shared__ Partial warp_part[kResidualWarps];
    __shared__ Partial cta_part[kSmallMaxCtasPerRow];  // (used in the row's first CTA)
    const int b = blockIdx.y, part = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), G.K) : G.K;
    cudaGridDependencySynchronize();  // an earlier call on the stream may still be reading the partials

    const int rows = G.K * G.units_per_row;  // rows of the window that are streamed
    const int group = G.small_group;
    int r, seg, segs;  // this warp: row of the window, its segment of the row, segments per row
    if (group == kResidualWarps) {
        r = part / G.small_ctas_per_row;
        seg = (part - r * G.small_ctas_per_row) * kResidualWarps + warp;
        segs = G.small_ctas_per_row * kResidualWarps;
    } else {
        r = part * (kResidualWarps / group) + warp / group;
        seg = warp % group;
        segs = group;
    }
    RowState st;
    st.reset();
    const int i_row = G.units_per_row == 2 ? (r >> 1) : r;
    if (r < rows && i_row < n) {
        const bool is_draft = G.units_per_row == 2 && (r & 1);
        const int64_t row = static_cast<int64_t>(b) * G.K + i_row;
        const int nvec = G.vec_bytes / 16;
        const int v0 = static_cast<int>(static_cast<int64_t>(seg) * nvec / segs);
        const int v1 = static_cast<int>(static_cast<int64_t>(seg + 1) * nvec / segs);
        const char* base = (is_draft ? P.draft : P.target) + row * G.ld_bytes + static_cast<int64_t>(v0) * 16;
        const int len = (v1 - v0) * 16;
        constexpr int kBatchBytes = 32 * 16 * kVecPerThread;
        for (int off = 0; off < len; off += kSmallDepth * kBatchBytes) {
            uint4 w[kSmallDepth][kVecPerThread];
            int at[kSmallDepth][kVecPerThread];
#pragma unroll
            for (int h = 0; h < kSmallDepth; ++h)
#pragma unroll
                for (int j = 0; j < kVecPerThread; ++j) {
                    at[h][j] = off + h * kBatchBytes + j * 32 * 16 + lane * 16;
                    if (at[h][j] < len) w[h][j] = ld_global_nc_v4(base + at[h][j]);
                }
            if (st.ref == kNoReference && at[0][0] < len) st.ref = first_reference<DT>(w[0][0], P.c_hi, P.c_lo);
#pragma unroll
            for (int h = 0; h < kSmallDepth; ++h) {
                if (off + h * kBatchBytes >= len) break;  // uniform over the warp
                if (at[h][kVecPerThread - 1] < len)
                    absorb_tile<DT, true>(w[h], at[h], len, P.c_hi, P.c_lo, st);
                else
                    absorb_tile<DT, false>(w[h], at[h], len, P.c_hi, P.c_lo, st);
            }
        }
    }
    {
        const Partial mine = warp_combine<false>(st.ref, st.sum, st.best, st.index);
        if (lane == 0) warp_part[warp] = mine;
    }
    __syncthreads();
    Partial all;
    all.ref = kNoReference;
    all.sum = 0.f;
    all.best = -INFINITY;
    all.index = 0x7FFFFFFF;
    if (warp < kResidualWarps / group) {  // warp g folds the records of the g-th group of warps
        if (lane < group) all = warp_part[warp * group + lane];
        all = warp_combine<false>(all.ref, all.sum, all.best, all.index);
    }
    if constexpr (CLUSTER) {
        // whole CTAs share the row: their records go to the first one, which folds them
        const int rank = part % G.small_ctas_per_row;
        if (threadIdx.x == 0) cg::this_cluster().map_shared_rank(cta_part, 0)[rank] = all;
        cg::this_cluster().sync();
        if (rank == 0 && warp == 0) {
            Partial rec;
            rec.ref = kNoReference;
            rec.sum = 0.f;
            rec.best = -INFINITY;
            rec.index = 0x7FFFFFFF;
            if (lane < G.small_ctas_per_row) rec = cta_part[lane];
            rec = warp_combine<false>(rec.ref, rec.sum, rec.best, rec.index);
            if (lane == 0 && r < rows) P.partials[static_cast<int64_t>(b) * rows + r] = rec;
        }
    } else if (warp < kResidualWarps / group) {
        const int rg = group == kResidualWarps ? part : part * (kResidualWarps / group) + warp;
        if (lane == 0 && rg < rows) P.partials[static_cast<int64_t>(b) * rows + rg] = all;
    }
}

// =================================================== vocabulary-parallel ====
// The same verification when the vocabulary axis is split over ranks (logits leaving a
// tensor-parallel LM head): every rank streams its slice once, the ranks exchange six numbers
// per position, decide the acceptance tests identically, draw their share of each residual
// sample over their slice and exchange one candidate per rejected window.
constexpr int kVpStatsPerRow = 6;  // M_p, S_p, M_q, S_q, l^p[x], l^q[x]

// Per row of this rank's slice: the (reference, sum) pairs of the two laws and, on the rank whose
// slice holds the draft token, the two logits at it (NaN elsewhere).  S = NaN marks bad data.
template <int DT>
__global__ void __launch_bounds__(128) vp_stats_kernel(const __grid_constant__ VerifyParams P, double* __restrict__ stats) {
    const Geometry& G = P.geo;
    cudaGridDependencySynchronize();  // the streaming kernel's partials must be complete and visible
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= static_cast<int64_t>(G.B) * G.K) return;
    const int b = static_cast<int>(row / G.K), i = static_cast<int>(row - static_cast<int64_t>(b) * G.K);
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), G.K) : G.K;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);
    const double nan = __longlong_as_double(0x7FF8000000000000ll);
    double out[kVpStatsPerRow] = {-INFINITY, 0.0, -INFINITY, 0.0, nan, nan};
    if (i < n) {
        const char* prow = P.target + row * G.ld_bytes;
        const char* qrow = P.draft + row * G.ld_bytes;
        const RowNorm np = fold_unit<DT, false>(2 * row, prow, c, P);
        const RowNorm nq = fold_unit<DT, false>(2 * row + 1, qrow, c, P);
        out[0] = np.M;
        out[1] = np.data_bad ? nan : np.S;
        out[2] = nq.M;
        out[3] = nq.data_bad ? nan : nq.S;
        const int x = __ldg(P.draft_tokens + row) - P.vocab_offset;
        if (x >= 0 && x < G.V) {
            out[4] = load_logit<DT>(prow, x);
            out[5] = load_logit<DT>(qrow, x);
        }
    }
#pragma unroll
    for (int k = 0; k < kVpStatsPerRow; ++k) stats[row * kVpStatsPerRow + k] = out[k];
}

// The ranks' (reference, sum) pairs of one law folded into its log2 normaliser; false on bad data.
__device__ bool vp_fold(const double* __restrict__ stats, int ranks, int64_t rows, int64_t row, int at, double* k_out) {
    double M = -INFINITY, S = 0.0;
    bool bad = false;
    for (int r = 0; r < ranks; ++r) {
        const double* rec = stats + (static_cast<int64_t>(r) * rows + row) * kVpStatsPerRow + at;
        const double m = rec[0], sum = rec[1];
        if (!(sum >= 0.0) || sum == INFINITY) bad = true;
        if (sum > 0.0) {
            if (m > M) {
                S = S * exp2(M - m) + sum;
                M = m;
            } else {
                S += sum * exp2(m - M);
            }
        }
    }
    if (bad || !(S > 0.0) || !(S < INFINITY)) return false;
    *k_out = M + log2(S);
    return true;
}

// Acceptance tests, first rejection and outputs from the gathered statistics: one CTA per
// window, one thread per position; every rank runs it on the same numbers.
__global__ void __launch_bounds__(FEF_MAX_K) vp_accept_kernel(const __grid_constant__ VerifyParams P,
                                                              const double* __restrict__ stats, int ranks, int V_total) {
    const Geometry& G = P.geo;
    const int b = blockIdx.x, i = threadIdx.x;
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), G.K) : G.K;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);
    const int64_t rows = static_cast<int64_t>(G.B) * G.K, row = static_cast<int64_t>(b) * G.K + i;
    __shared__ int s_accept[FEF_MAX_K], s_err[FEF_MAX_K];
    __shared__ double s_kp[FEF_MAX_K], s_kq[FEF_MAX_K];
    int tok = -1;
    float conf = -1.f;
    if (i < n) {
        int err = 0, accept = 0;
        double kp = 0.0, kq = 0.0;
        tok = __ldg(P.draft_tokens + row);
        double lpx = 0.0, lqx = 0.0;
        int owners = 0;
        for (int r = 0; r < ranks; ++r) {
            const double* rec = stats + (static_cast<int64_t>(r) * rows + row) * kVpStatsPerRow;
            if (rec[4] == rec[4]) {  // not NaN: this rank holds the token
                lpx = rec[4];
                lqx = rec[5];
                ++owners;
            }
        }
        if (tok < 0 || tok >= V_total || owners != 1) {
            err = FEF_ERR_TOKEN_RANGE;
        } else if (!vp_fold(stats, ranks, rows, row, 0, &kp) || !vp_fold(stats, ranks, rows, row, 2, &kq)) {
            err = FEF_ERR_NONFINITE;
        } else {
            const double l2pi = lpx * c - kp;  // log2 pi(x)
            conf = static_cast<float>(exp2(l2pi));
            if (lqx == -INFINITY) {
                accept = lpx > -INFINITY;  // rho(x) = 0: accept iff pi(x) > 0
            } else {
                const double ratio = exp2(l2pi - (lqx * c - kq));
                const uint4 r = philox4x32_10(
                    make_uint4(kStreamAccept << 30, static_cast<uint32_t>(b), static_cast<uint32_t>(i), step_of(P)),
                    make_uint2(static_cast<uint32_t>(P.seed), static_cast<uint32_t>(P.seed >> 32)));
                accept = static_cast<double>(uniform_from_word(r.x)) <= fmin(1.0, ratio);
            }
        }
        s_err[i] = err;
        s_accept[i] = accept;
        s_kp[i] = kp;
        s_kq[i] = kq;
    }
    __syncthreads();
    int err = 0, a = n;
    for (int k = 0; k < n; ++k) err = max(err, s_err[k]);
    for (int k = n - 1; k >= 0; --k)
        if (!s_accept[k]) a = k;
    if (i < G.K) {
        const bool keep = !err && i < a;
        P.tokens[row] = keep ? tok : -1;
        P.conf[row] = keep ? conf : -1.f;
    }
    if (i == 0) {
        P.accept_len[b] = err ? -1 : a;
        if (err) report(P.status, err);
        ResidualTask task;
        task.pos = (!err && a < n) ? a : -1;
        task.arrivals = 0u;
        task.kp = task.pos >= 0 ? s_kp[a] : 0.0;
        task.kq = task.pos >= 0 ? s_kq[a] : 0.0;
        P.tasks[b] = task;
    }
}

// The ranks' candidates of each rejected window compared: the largest exact score wins (lowest
// id on ties); if no rank has a positive residual weight, the largest target logit does.
__global__ void __launch_bounds__(128) vp_finish_kernel(const __grid_constant__ VerifyParams P,
                                                        const VpCandidate* __restrict__ cands, int ranks) {
    const Geometry& G = P.geo;
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= G.B) return;
    const ResidualTask task = P.tasks[b];
    if (task.pos < 0) return;
    const double c = static_cast<double>(P.c_hi) + static_cast<double>(P.c_lo);
    double best = -INFINITY;
    float best_lp = -INFINITY, lp = 0.f;
    int Z = 0x7FFFFFFF, Zl = 0x7FFFFFFF;
    for (int r = 0; r < ranks; ++r) {
        const VpCandidate cd = cands[static_cast<int64_t>(r) * G.B + b];
        if (cd.score > best || (cd.score == best && cd.score > -INFINITY && cd.index < Z)) {
            best = cd.score;
            Z = cd.index;
            lp = cd.lp;
        }
        if (cd.lp > best_lp || (cd.lp == best_lp && cd.index < Zl)) {
            best_lp = cd.lp;
            Zl = cd.index;
        }
    }
    if (!(best > -INFINITY)) {  // [pi - rho]_+ is zero everywhere: arg-max of pi
        Z = Zl;
        lp = best_lp;
    }
    const int64_t row = static_cast<int64_t>(b) * G.K + task.pos;
    P.tokens[row] = Z;
    P.conf[row] = static_cast<float>(exp2(static_cast<double>(lp) * c - task.kp));
}

// ================================================================= host ====
static int g_sm_count[64];
static bool g_attr_done[64][4];

constexpr int kClaimsPerCta = 3;             // streaming claims a CTA should get at least, size permitting (6 cost B = 1 calls 4 us)
constexpr int kMaxClaimBytes = 1 << 20;      // and at most this many bytes per claim (a whole row of the usual sizes)

static int sm_count_of_current_device(int* device_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (g_sm_count[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        g_sm_count[dev] = n;
    }
    if (device_out) *device_out = dev;
    return g_sm_count[dev];
}


// small_capacity: CTAs of small_rows_kernel the device holds at once when the call may take the path for
// few rows (sampling mode, the target rows streamed, no timing marks), else 0.
static bool make_geometry(int B, int K, int V, int64_t ld, fef_dtype dt, bool target_only, int sm_count,
                          Geometry* out, int small_capacity = 0) {
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V < 1 || ld < V || sm_count < 1) return false;
    if (dt != FEF_F32 && dt != FEF_BF16) return false;
    const int esize = dt == FEF_F32 ? 4 : 2;
    if (static_cast<int64_t>(V) * esize > (1ll << 30)) return false;
    Geometry G;
    G.B = B;
    G.K = K;
    G.V = V;
    G.units_per_row = target_only ? 1 : 2;
    G.ld_bytes = ld * esize;
    G.vec_bytes = static_cast<int>((static_cast<int64_t>(V) * esize) / 16 * 16);
    G.vec_elems = G.vec_bytes / esize;
    G.num_units = static_cast<int64_t>(B) * K * G.units_per_row;

    // streaming claims: large enough to amortise their bookkeeping, small enough that every
    // CTA gets several and the last ones end close together
    int64_t claim_target = G.num_units * G.vec_bytes / (static_cast<int64_t>(sm_count) * kClaimsPerCta);
    if (claim_target > kMaxClaimBytes) claim_target = kMaxClaimBytes;
    if (claim_target < 8192) claim_target = 8192;
    G.tile_bytes = kTileBytes;
    while (G.tile_bytes > 8192 && G.tile_bytes > claim_target) G.tile_bytes >>= 1;
    G.tiles_per_unit = (G.vec_bytes + G.tile_bytes - 1) / G.tile_bytes;
    if (G.tiles_per_unit > 0) {
        int tpc = static_cast<int>(claim_target / G.tile_bytes);
        if (tpc < 1) tpc = 1;
        if (tpc > G.tiles_per_unit) tpc = G.tiles_per_unit;
        G.claims_per_unit = (G.tiles_per_unit + tpc - 1) / tpc;
        G.tiles_per_claim = (G.tiles_per_unit + G.claims_per_unit - 1) / G.claims_per_unit;  // even split
        G.claims_per_unit = (G.tiles_per_unit + G.tiles_per_claim - 1) / G.tiles_per_claim;
    } else {
        G.tiles_per_claim = 1;
        G.claims_per_unit = 1;
    }
    G.num_claims = G.num_units * G.claims_per_unit;
    if (G.num_claims >= (1ll << 31)) return false;  // claim numbers are handled as 32-bit values
    G.grid = static_cast<int>(G.num_claims < sm_count ? G.num_claims : sm_count);
    // Rows of at most one tile, enough of them to give every resident warp its own: the ring would
    // end every tile in a cross-warp combine, so a warp takes a whole row instead
    G.warp_per_row = (G.vec_bytes > 0 && G.vec_bytes <= kTileBytes &&
                      G.num_units >= static_cast<int64_t>(sm_count) * kRowsWarps * 2) ? 1 : 0;
    if (G.warp_per_row) {
        G.claims_per_unit = 1;
        G.num_claims = G.num_units;
        const int64_t ctas = (G.num_units + kRowsWarps - 1) / kRowsWarps;
        const int64_t cap = static_cast<int64_t>(sm_count) * kRowsCtasPerSm;
        G.grid = static_cast<int>(ctas < cap ? ctas : cap);
    }

    // residual kernel: CTAs per rejected row, each thread up to kResidualBatch vector pairs
    // (fewer when few windows would leave SMs idle)
    const int nvec = G.vec_bytes / 16;
    int per_thread = 4;
    while (per_thread > 1 &&
           static_cast<int64_t>(B) * ((nvec + kResidualThreads * per_thread - 1) / (kResidualThreads * per_thread)) < 2 * sm_count)
        per_thread >>= 1;
    int parts = (nvec + kResidualThreads * per_thread - 1) / (kResidualThreads * per_thread);
    // all CTAs of the call resident at once (kResidualCtasPerSm per SM) where that is possible: one
    // wave of CTAs that loop beats several waves of CTAs that each pay the start-up latencies
    const int resident = (kResidualCtasPerSm * sm_count) / B;
    if (resident >= 1 && parts > resident) parts = resident;
    if (parts > kMaxResidualCtas) parts = kMaxResidualCtas;
    if (parts < 1) parts = 1;
    G.residual_ctas = parts;

    // few rows: the window's CTAs split its rows by groups of warps
    G.small = 0;
    G.small_parts = 0;
    G.small_group = 0;
    G.small_ctas_per_row = 0;
    if (small_capacity > kMaxSmallCtas) small_capacity = kMaxSmallCtas;
    const int small_parts = small_capacity / B;
    const int rows = K * G.units_per_row;
    if (small_parts >= 1 && G.vec_bytes > 0 && G.num_units * G.vec_bytes <= kSmallMaxBytes &&
        small_parts * kResidualWarps >= rows) {
        const int warps_per_row = small_parts * kResidualWarps / rows;
        G.small = 1;
        if (warps_per_row >= kResidualWarps) {
            G.small_group = kResidualWarps;
            G.small_ctas_per_row = warps_per_row / kResidualWarps;
            if (G.small_ctas_per_row > kSmallMaxCtasPerRow) G.small_ctas_per_row = kSmallMaxCtasPerRow;
        } else {
            G.small_group = warps_per_row >= 4 ? 4 : warps_per_row >= 2 ? 2 : 1;
            G.small_ctas_per_row = 1;
        }
        G.claims_per_unit = 1;
        G.num_claims = G.num_units;
        // as many CTAs as have a row to work on
        G.small_parts = G.small_group == kResidualWarps ? rows * G.small_ctas_per_row
                                                         : (rows * G.small_group + kResidualWarps - 1) / kResidualWarps;
        G.warp_per_row = 0;
    }
    *out = G;
    return true;
}

// Scratch layout: control (cleared on every call), partials, tasks, candidates (every value
// written before it is read).
struct WorkspaceLayout {
    size_t control, zero_bytes, partials, tasks, candidates, total;
};
static size_t round256(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }
static WorkspaceLayout layout_of(const Geometry& G) {
    WorkspaceLayout L;
    L.control = 0;
    L.zero_bytes = round256(sizeof(Control));
    L.partials = L.zero_bytes;
    L.tasks = L.partials + round256(static_cast<size_t>(G.num_claims) * sizeof(Partial));
    L.candidates = L.tasks + round256(static_cast<size_t>(G.B) * sizeof(ResidualTask));
    L.total = L.candidates + round256(static_cast<size_t>(G.B) * kMaxResidualCtas * kCandidatesPerCta * sizeof(Candidate));
    return L;
}

// Launch with programmatic dependent launch: the grid may be scheduled while its
// predecessor on the stream drains; the kernel itself waits (cudaGridDependencySynchronize)
// before touching anything the predecessor wrote.
template <typename... Args>
static cudaError_t launch_dependent(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
// The same with the CTAs of a grid row (blockIdx.y) grouped into one thread-block cluster.
template <typename... Args>
static cudaError_t launch_dependent_cluster(int cluster_x, void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem,
                                            cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = static_cast<unsigned>(cluster_x);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

static void mark(void* const* events, int which, cudaStream_t stream) {
    if (events && events[which]) cudaEventRecord(static_cast<cudaEvent_t>(events[which]), stream);
}

// events (may be null): [0] before the streaming kernel, [1] after it, [2] and [3] after the kernel
// that follows it (sampling mode: acceptance tests and residual draw in one launch; greedy mode: the scan)
template <int DT, bool GREEDY>
static cudaError_t launch_all(const VerifyParams& P, int dev, cudaStream_t stream, void* const* events) {
    const Geometry& G = P.geo;
    const int which = DT * 2 + (GREEDY ? 1 : 0);
    if (!g_attr_done[dev][which]) {
        const cudaError_t e = cudaFuncSetAttribute(stream_kernel<DT, GREEDY>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        g_attr_done[dev][which] = true;
    }
    cudaError_t e;
    if constexpr (!GREEDY) {
        if (G.small) {
            // few rows: the latency-oriented kernel streams instead
            e = launch_dependent(begin_call_kernel, dim3(1), dim3(kBeginThreads), 0, stream, P.ctl, P.tasks, G.B, P.status);
            if (e != cudaSuccess) return e;
            if (G.small_ctas_per_row > 1)
                e = launch_dependent_cluster(G.small_ctas_per_row, small_rows_kernel<DT, true>, dim3(G.small_parts, G.B),
                                             dim3(kResidualThreads), 0, stream, P);
            else
                e = launch_dependent(small_rows_kernel<DT, false>, dim3(G.small_parts, G.B), dim3(kResidualThreads), 0,
                                     stream, P);
            if (e != cudaSuccess) return e;
            if (G.residual_ctas <= kMaxClusterCtas)
                e = launch_dependent_cluster(G.residual_ctas, tail_kernel<DT, true>, dim3(G.residual_ctas, G.B),
                                             dim3(kResidualThreads), 0, stream, P);
            else
                e = launch_dependent(tail_kernel<DT, false>, dim3(G.residual_ctas, G.B), dim3(kResidualThreads), 0, stream, P);
            if (e != cudaSuccess) return e;
            return cudaGetLastError();
        }
    }
    if (!GREEDY && P.target_norm) {
        // both laws' normalisers are given: only the counters are cleared, then the last kernel runs
        e = launch_dependent(begin_call_kernel, dim3(1), dim3(kBeginThreads), 0, stream, P.ctl, P.tasks, G.B, P.status);
        if (e != cudaSuccess) return e;
    } else if (events) {
        // timing marks asked for: clear with memset nodes and launch the streaming kernel the
        // ordinary way, so that the first two marks bracket that kernel alone
        if (P.status && (e = cudaMemsetAsync(P.status, 0, sizeof(int32_t), stream)) != cudaSuccess) return e;
        if ((e = cudaMemsetAsync(P.ctl, 0, sizeof(Control), stream)) != cudaSuccess) return e;
        if ((e = cudaMemsetAsync(P.tasks, 0, sizeof(ResidualTask) * G.B, stream)) != cudaSuccess) return e;
        mark(events, 0, stream);
        if (G.warp_per_row)
            rows_kernel<DT, GREEDY><<<G.grid, kRowsWarps * 32, 0, stream>>>(P);
        else
            stream_kernel<DT, GREEDY><<<G.grid, kStreamThreads, kSmemBytes, stream>>>(P);
    } else {
        e = launch_dependent(begin_call_kernel, dim3(1), dim3(kBeginThreads), 0, stream, P.ctl, P.tasks, G.B, P.status);
        if (e != cudaSuccess) return e;
        if (G.warp_per_row)
            e = launch_dependent(rows_kernel<DT, GREEDY>, dim3(G.grid), dim3(kRowsWarps * 32), 0, stream, P);
        else
            e = launch_dependent(stream_kernel<DT, GREEDY>, dim3(G.grid), dim3(kStreamThreads), kSmemBytes, stream, P);
        if (e != cudaSuccess) return e;
    }
    mark(events, 1, stream);
    if constexpr (GREEDY) {
        if (G.claims_per_unit >= 4)  // few rows, many partials per row: one warp per position
            e = launch_dependent(scan_rows_kernel<DT>, dim3(G.B), dim3(32 * (G.K < kScanMaxWarps ? G.K : kScanMaxWarps)), 0,
                                 stream, P);
        else
            e = launch_dependent(scan_kernel<DT>, dim3((G.B + kScanWarps - 1) / kScanWarps), dim3(kScanWarps * 32), 0,
                                 stream, P);
    } else {
        if (G.residual_ctas <= kMaxClusterCtas)
            e = launch_dependent_cluster(G.residual_ctas, tail_kernel<DT, true>, dim3(G.residual_ctas, G.B),
                                         dim3(kResidualThreads), 0, stream, P);
        else
            e = launch_dependent(tail_kernel<DT, false>, dim3(G.residual_ctas, G.B), dim3(kResidualThreads), 0, stream, P);
    }
    if (e != cudaSuccess) return e;
    mark(events, 2, stream);
    mark(events, 3, stream);
    return cudaGetLastError();
}

}  // namespace fef

extern "C" {

const char* fef_status_string(fef_status s) {
    switch (s) {
        case FEF_OK: return "ok";
        case FEF_ERR_INVALID_ARG: return "invalid argument";
        case FEF_ERR_DTYPE: return "unsupported dtype";
        case FEF_ERR_ALIGNMENT: return "logit pointer or row pitch not a multiple of 16 bytes";
        case FEF_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case FEF_ERR_CUDA: return "CUDA error or no CUDA device";
        case FEF_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case FEF_ERR_NONFINITE: return "NaN or +inf logit, or a row of -inf only";
        case FEF_ERR_TOKEN_RANGE: return "draft token outside [0, V)";
        case FEF_ERR_TOO_LARGE: return "sizes need more scratch than the built-in buffer of fef_spec_verify_static holds";
    }
    return "unknown status";
}

size_t fef_spec_verify_workspace_bytes(int B, int K, int V, fef_dtype dt) {
    const int sms = fef::sm_count_of_current_device(nullptr);
    fef::Geometry sampling, greedy;
    if (!fef::make_geometry(B, K, V, V, dt, false, sms, &sampling)) return 0;
    if (!fef::make_geometry(B, K, V, V, dt, true, sms, &greedy)) return 0;
    size_t need = fef::layout_of(sampling).total;  // one buffer serves every mode
    const size_t g = fef::layout_of(greedy).total;
    if (g > need) need = g;
    const int capacity = fef::kResidualCtasPerSm * sms;
    for (int target_only = 0; target_only < 2 && capacity > 0; ++target_only) {
        fef::Geometry few_rows;
        if (!fef::make_geometry(B, K, V, V, dt, target_only != 0, sms, &few_rows, capacity)) return 0;
        const size_t s = fef::layout_of(few_rows).total;
        if (s > need) need = s;
    }
    return need;
}

}  // extern "C"

#ifdef FEF_TEST_HOOKS
// Test builds only (never part of the shipped library): the next verification call makes the
// streaming kernel's CTA 0 withhold its stage number `stage` and lets waits give up after
// `limit_ns`, so that the give-up path can be exercised without faulting or hanging anything.
static int g_test_withhold_stage = -1;
static unsigned long long g_test_wait_limit_ns = 0;
extern "C" void fef_test_withhold_stage_once(int stage, unsigned long long limit_ns) {
    g_test_withhold_stage = stage;
    g_test_wait_limit_ns = limit_ns;
}
#endif

// Every verification entry point ends here.
static fef_status verify_impl(const void* draft_logits, const void* target_logits, const int32_t* draft_tokens,
                              const int32_t* row_len, const double* draft_log2_norm, int B, int K, int V, int64_t ld,
                              fef_dtype dt, float temperature, uint64_t seed, uint32_t step, int32_t* accept_len,
                              int32_t* tokens, float* conf, void* workspace, size_t workspace_bytes,
                              int32_t* device_status, void* cuda_stream, void* const* stage_events,
                              const uint32_t* device_round = nullptr, const double* target_log2_norm = nullptr) {
    using namespace fef;
    if (dt != FEF_F32 && dt != FEF_BF16) return FEF_ERR_DTYPE;
    if (!draft_logits || !target_logits || !draft_tokens || !accept_len || !tokens || !conf)
        return FEF_ERR_INVALID_ARG;
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V < 1 || ld < V) return FEF_ERR_INVALID_ARG;
    if (!(temperature >= 0.0f) || isinf(temperature)) return FEF_ERR_INVALID_ARG;
    const int esize = dt == FEF_F32 ? 4 : 2;
    if (static_cast<int64_t>(V) * esize > (1ll << 30)) return FEF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(draft_logits) & 15) || (reinterpret_cast<uintptr_t>(target_logits) & 15) ||
        ((ld * esize) & 15))
        return FEF_ERR_ALIGNMENT;

    int dev = 0;
    const int sms = sm_count_of_current_device(&dev);
    if (sms < 1) return FEF_ERR_CUDA;
    const bool greedy = (temperature == 0.0f);

    VerifyParams P;
    // the path for few rows: sampling mode with the target rows to stream, no timing marks
    const bool small_ok = !greedy && !stage_events && !(draft_log2_norm && target_log2_norm);
    if (!make_geometry(B, K, V, ld, dt, greedy || draft_log2_norm != nullptr, sms, &P.geo,
                       small_ok ? kResidualCtasPerSm * sms : 0))
        return FEF_ERR_INVALID_ARG;
    const WorkspaceLayout L = layout_of(P.geo);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < L.total)
        return FEF_ERR_WORKSPACE;

    // c = log2(e) / T (greedy mode reports T = 1 confidences).  binary32 logits: c = c_hi + c_lo
    // with c_lo > 0, applied with two fused multiply-adds.  bfloat16 logits: the nearest binary32
    // number alone (c_lo = 0), i.e. the softmax is evaluated at T (1 + d) with |d| <= 6e-8.
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
    P.c_exact = c;
    if (!(P.c_hi > 0.f) || isinf(P.c_hi)) return FEF_ERR_INVALID_ARG;
    P.wait_limit_ns = kWaitLimitNs;
    P.withhold_stage = -1;
#ifdef FEF_TEST_HOOKS
    if (g_test_withhold_stage >= 0) {  // one call only
        P.withhold_stage = g_test_withhold_stage;
        P.wait_limit_ns = g_test_wait_limit_ns;
        g_test_withhold_stage = -1;
    }
#endif

    P.target = static_cast<const char*>(target_logits);
    P.draft = static_cast<const char*>(draft_logits);
    P.draft_tokens = draft_tokens;
    P.row_len = row_len;
    P.draft_norm = greedy ? nullptr : draft_log2_norm;
    P.target_norm = (greedy || !draft_log2_norm) ? nullptr : target_log2_norm;
    P.seed = seed;
    P.keys = philox_round_keys(seed);
    P.step = step;
    P.round = device_round;
    P.accept_len = accept_len;
    P.tokens = tokens;
    P.conf = conf;
    char* ws = static_cast<char*>(workspace);
    P.ctl = reinterpret_cast<Control*>(ws + L.control);
    P.partials = reinterpret_cast<Partial*>(ws + L.partials);
    P.tasks = reinterpret_cast<ResidualTask*>(ws + L.tasks);
    P.candidates = reinterpret_cast<Candidate*>(ws + L.candidates);
    P.vocab_offset = 0;
    P.vp_out = nullptr;
    P.status = device_status;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the call's first kernel clears the claim counter and the status word; nothing else in the
    // scratch needs a defined value
    cudaError_t e;
    if (dt == FEF_F32)
        e = greedy ? launch_all<FEF_F32, true>(P, dev, stream, stage_events)
                   : launch_all<FEF_F32, false>(P, dev, stream, stage_events);
    else
        e = greedy ? launch_all<FEF_BF16, true>(P, dev, stream, stage_events)
                   : launch_all<FEF_BF16, false>(P, dev, stream, stage_events);
    return e == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

extern "C" {

fef_status fef_spec_verify_profiled(const void* draft_logits, const void* target_logits,
                                    const int32_t* draft_tokens, const int32_t* row_len, int B, int K, int V,
                                    int64_t ld, fef_dtype dt, float temperature, uint64_t seed, uint32_t step,
                                    int32_t* accept_len, int32_t* tokens, float* conf, void* workspace,
                                    size_t workspace_bytes, int32_t* device_status, void* cuda_stream,
                                    void* const* stage_events) {
    return verify_impl(draft_logits, target_logits, draft_tokens, row_len, nullptr, B, K, V, ld, dt, temperature, seed,
                       step, accept_len, tokens, conf, workspace, workspace_bytes, device_status, cuda_stream,
                       stage_events);
}

fef_status fef_spec_verify(const void* draft_logits, const void* target_logits, const int32_t* draft_tokens,
                           const int32_t* row_len, int B, int K, int V, int64_t ld, fef_dtype dt,
                           float temperature, uint64_t seed, uint32_t step, int32_t* accept_len,
                           int32_t* tokens, float* conf, void* workspace, size_t workspace_bytes,
                           int32_t* device_status, void* cuda_stream) {
    return verify_impl(draft_logits, target_logits, draft_tokens, row_len, nullptr, B, K, V, ld, dt, temperature, seed,
                       step, accept_len, tokens, conf, workspace, workspace_bytes, device_status, cuda_stream, nullptr);
}

fef_status fef_spec_verify_with_draft_norm(const void* draft_logits, const void* target_logits,
                                           const int32_t* draft_tokens, const double* draft_log2_norm,
                                           const int32_t* row_len, int B, int K, int V, int64_t ld, fef_dtype dt,
                                           float temperature, uint64_t seed, uint32_t step, int32_t* accept_len,
                                           int32_t* tokens, float* conf, void* workspace, size_t workspace_bytes,
                                           int32_t* device_status, void* cuda_stream) {
    if (!draft_log2_norm) return FEF_ERR_INVALID_ARG;
    return verify_impl(draft_logits, target_logits, draft_tokens, row_len, draft_log2_norm, B, K, V, ld, dt,
                       temperature, seed, step, accept_len, tokens, conf, workspace, workspace_bytes, device_status,
                       cuda_stream, nullptr);
}

fef_status fef_spec_verify_with_norms(const void* draft_logits, const void* target_logits, const int32_t* draft_tokens,
                                      const double* draft_log2_norm, const double* target_log2_norm,
                                      const int32_t* row_len, int B, int K, int V, int64_t ld, fef_dtype dt,
                                      float temperature, uint64_t seed, uint32_t step, const uint32_t* device_round,
                                      int32_t* accept_len, int32_t* tokens, float* conf, void* workspace,
                                      size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    if (!draft_log2_norm || !target_log2_norm) return FEF_ERR_INVALID_ARG;
    return verify_impl(draft_logits, target_logits, draft_tokens, row_len, draft_log2_norm, B, K, V, ld, dt,
                       temperature, seed, step, accept_len, tokens, conf, workspace, workspace_bytes, device_status,
                       cuda_stream, nullptr, device_round, target_log2_norm);
}

fef_status fef_spec_verify_at_round(const void* draft_logits, const void* target_logits,
                                    const int32_t* draft_tokens, const double* draft_log2_norm,
                                    const int32_t* row_len, int B, int K, int V, int64_t ld, fef_dtype dt,
                                    float temperature, uint64_t seed, uint32_t step, const uint32_t* device_round,
                                    int32_t* accept_len, int32_t* tokens, float* conf, void* workspace,
                                    size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    if (!device_round) return FEF_ERR_INVALID_ARG;
    return verify_impl(draft_logits, target_logits, draft_tokens, row_len, draft_log2_norm, B, K, V, ld, dt,
                       temperature, seed, step, accept_len, tokens, conf, workspace, workspace_bytes, device_status,
                       cuda_stream, nullptr, device_round);
}

}  // extern "C"

// Parameter block of a vocabulary-parallel call on this rank's slice (no launch).
static fef_status vp_setup(const void* draft_slice, const void* target_slice, const int32_t* draft_tokens,
                           const int32_t* row_len, int B, int K, int V_local, int64_t ld, fef_dtype dt,
                           float temperature, uint64_t seed, uint32_t step, int vocab_offset, void* workspace,
                           size_t workspace_bytes, bool need_logits, fef::VerifyParams* out, int* dev_out) {
    using namespace fef;
    if (dt != FEF_F32 && dt != FEF_BF16) return FEF_ERR_DTYPE;
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V_local < 1 || ld < V_local) return FEF_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || isinf(temperature)) return FEF_ERR_INVALID_ARG;  // sampling mode only
    if (vocab_offset < 0 || (vocab_offset & 7)) return FEF_ERR_INVALID_ARG;
    const int esize = dt == FEF_F32 ? 4 : 2;
    if (static_cast<int64_t>(V_local) * esize > (1ll << 30)) return FEF_ERR_INVALID_ARG;
    if (need_logits) {
        if (!draft_slice || !target_slice) return FEF_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(draft_slice) & 15) || (reinterpret_cast<uintptr_t>(target_slice) & 15) ||
            ((ld * esize) & 15))
            return FEF_ERR_ALIGNMENT;
    }
    const int sms = sm_count_of_current_device(dev_out);
    if (sms < 1) return FEF_ERR_CUDA;
    VerifyParams P = {};
    if (!make_geometry(B, K, V_local, ld, dt, false, sms, &P.geo)) return FEF_ERR_INVALID_ARG;
    const double c = 1.4426950408889634074 / static_cast<double>(temperature);
    float c_hi = static_cast<float>(c);
    if (dt == FEF_F32) {
        if (static_cast<double>(c_hi) >= c) c_hi = nextafterf(c_hi, 0.0f);
        P.c_lo = static_cast<float>(c - static_cast<double>(c_hi));
        if (!(P.c_lo > 0.f)) return FEF_ERR_INVALID_ARG;
    }
    P.c_hi = c_hi;
    P.c_exact = c;
    if (!(P.c_hi > 0.f) || isinf(P.c_hi)) return FEF_ERR_INVALID_ARG;
    P.wait_limit_ns = kWaitLimitNs;
    P.withhold_stage = -1;
    P.target_norm = nullptr;
    P.target = static_cast<const char*>(target_slice);
    P.draft = static_cast<const char*>(draft_slice);
    P.draft_tokens = draft_tokens;
    P.row_len = row_len;
    P.seed = seed;
    P.keys = philox_round_keys(seed);
    P.step = step;
    P.vocab_offset = vocab_offset;
    if (workspace) {
        const WorkspaceLayout L = layout_of(P.geo);
        if ((reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < L.total) return FEF_ERR_WORKSPACE;
        char* ws = static_cast<char*>(workspace);
        P.ctl = reinterpret_cast<Control*>(ws + L.control);
        P.partials = reinterpret_cast<Partial*>(ws + L.partials);
        P.candidates = reinterpret_cast<Candidate*>(ws + L.candidates);
    }
    *out = P;
    return FEF_OK;
}

template <int DT>
static cudaError_t vp_launch_stats(const fef::VerifyParams& P, int dev, double* stats, cudaStream_t stream) {
    using namespace fef;
    const Geometry& G = P.geo;
    const int which = DT * 2;
    if (!g_attr_done[dev][which]) {
        const cudaError_t e = cudaFuncSetAttribute(stream_kernel<DT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   static_cast<int>(kSmemBytes));
        if (e != cudaSuccess) return e;
        g_attr_done[dev][which] = true;
    }
    cudaError_t e;
    if (G.warp_per_row) {
        if (P.status && (e = cudaMemsetAsync(P.status, 0, sizeof(int32_t), stream)) != cudaSuccess) return e;
        e = launch_dependent(rows_kernel<DT, false>, dim3(G.grid), dim3(kRowsWarps * 32), 0, stream, P);
    } else {
        e = launch_dependent(begin_call_kernel, dim3(1), dim3(kBeginThreads), 0, stream, P.ctl,
                             static_cast<ResidualTask*>(nullptr), 0, P.status);
        if (e != cudaSuccess) return e;
        e = launch_dependent(stream_kernel<DT, false>, dim3(G.grid), dim3(kStreamThreads), kSmemBytes, stream, P);
    }
    if (e != cudaSuccess) return e;
    const int64_t rows = static_cast<int64_t>(G.B) * G.K;
    return launch_dependent(vp_stats_kernel<DT>, dim3(static_cast<unsigned>((rows + 127) / 128)), dim3(128), 0, stream, P,
                            stats);
}

extern "C" {

size_t fef_vp_task_bytes(int B) { return B < 1 ? 0 : static_cast<size_t>(B) * sizeof(fef::ResidualTask); }

fef_status fef_vp_local_stats(const void* draft_slice, const void* target_slice, const int32_t* draft_tokens,
                              const int32_t* row_len, int B, int K, int V_local, int64_t ld, fef_dtype dt,
                              float temperature, int vocab_offset, double* stats, void* workspace,
                              size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    using namespace fef;
    if (!draft_tokens || !stats || !workspace) return FEF_ERR_INVALID_ARG;
    VerifyParams P;
    int dev = 0;
    const fef_status st = vp_setup(draft_slice, target_slice, draft_tokens, row_len, B, K, V_local, ld, dt, temperature,
                                   0, 0, vocab_offset, workspace, workspace_bytes, true, &P, &dev);
    if (st != FEF_OK) return st;
    P.status = device_status;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const cudaError_t e = dt == FEF_F32 ? vp_launch_stats<FEF_F32>(P, dev, stats, stream)
                                        : vp_launch_stats<FEF_BF16>(P, dev, stats, stream);
    return e == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_vp_accept(const double* stats_all, int ranks, const int32_t* draft_tokens, const int32_t* row_len,
                         int B, int K, int V_total, fef_dtype dt, float temperature, uint64_t seed, uint32_t step,
                         int32_t* accept_len, int32_t* tokens, float* conf, void* tasks, int32_t* device_status,
                         void* cuda_stream) {
    using namespace fef;
    if (!stats_all || ranks < 1 || ranks > 1024 || !draft_tokens || !accept_len || !tokens || !conf || !tasks ||
        V_total < 1)
        return FEF_ERR_INVALID_ARG;
    VerifyParams P;
    int dev = 0;
    // (the slice width only shapes the streaming geometry, which this step does not use)
    const fef_status st = vp_setup(nullptr, nullptr, draft_tokens, row_len, B, K, 8, 8, dt, temperature, seed, step, 0,
                                   nullptr, 0, false, &P, &dev);
    if (st != FEF_OK) return st;
    P.accept_len = accept_len;
    P.tokens = tokens;
    P.conf = conf;
    P.tasks = static_cast<ResidualTask*>(tasks);
    P.status = device_status;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (device_status && cudaMemsetAsync(device_status, 0, sizeof(int32_t), stream) != cudaSuccess) return FEF_ERR_CUDA;
    vp_accept_kernel<<<B, FEF_MAX_K, 0, stream>>>(P, stats_all, ranks, V_total);
    return cudaGetLastError() == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_vp_local_residual(const void* draft_slice, const void* target_slice, void* tasks, int B, int K,
                                 int V_local, int64_t ld, fef_dtype dt, float temperature, uint64_t seed,
                                 uint32_t step, int vocab_offset, void* candidates, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
    using namespace fef;
    if (!tasks || !candidates || !workspace) return FEF_ERR_INVALID_ARG;
    VerifyParams P;
    int dev = 0;
    const fef_status st = vp_setup(draft_slice, target_slice, nullptr, nullptr, B, K, V_local, ld, dt, temperature, seed,
                                   step, vocab_offset, workspace, workspace_bytes, true, &P, &dev);
    if (st != FEF_OK) return st;
    P.tasks = static_cast<ResidualTask*>(tasks);
    P.vp_out = static_cast<VpCandidate*>(candidates);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const dim3 grid(P.geo.residual_ctas, B);
    if (dt == FEF_F32)
        residual_kernel<FEF_F32><<<grid, kResidualThreads, 0, stream>>>(P);
    else
        residual_kernel<FEF_BF16><<<grid, kResidualThreads, 0, stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_vp_finish(const void* candidates_all, int ranks, const void* tasks, int B, int K, fef_dtype dt,
                         float temperature, int32_t* tokens, float* conf, void* cuda_stream) {
    using namespace fef;
    if (!candidates_all || ranks < 1 || ranks > 1024 || !tasks || !tokens || !conf) return FEF_ERR_INVALID_ARG;
    VerifyParams P;
    int dev = 0;
    const fef_status st = vp_setup(nullptr, nullptr, nullptr, nullptr, B, K, 8, 8, dt, temperature, 0, 0, 0, nullptr, 0,
                                   false, &P, &dev);
    if (st != FEF_OK) return st;
    P.tokens = tokens;
    P.conf = conf;
    P.tasks = static_cast<ResidualTask*>(const_cast<void*>(tasks));
    vp_finish_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        P, static_cast<const VpCandidate*>(candidates_all), ranks);
    return cudaGetLastError() == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

// ---- host-buffer variant: layout of the caller's device arena
namespace {
struct ArenaLayout {
    size_t q, p, tok, row_len, accept_len, tokens, conf, status, workspace, total;
};
size_t up256(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }
bool arena_layout(int B, int K, int V, int64_t ld, fef_dtype dt, ArenaLayout* L) {
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V < 1 || ld < V) return false;
    if (dt != FEF_F32 && dt != FEF_BF16) return false;
    const size_t ws = fef_spec_verify_workspace_bytes(B, K, V, dt);
    if (ws == 0) return false;
    const size_t logits = static_cast<size_t>(B) * K * ld * (dt == FEF_F32 ? 4 : 2);
    size_t at = 0;
    L->q = at; at += up256(logits);
    L->p = at; at += up256(logits);
    L->tok = at; at += up256(static_cast<size_t>(B) * K * 4);
    L->row_len = at; at += up256(static_cast<size_t>(B) * 4);
    L->accept_len = at; at += up256(static_cast<size_t>(B) * 4);
    L->tokens = at; at += up256(static_cast<size_t>(B) * K * 4);
    L->conf = at; at += up256(static_cast<size_t>(B) * K * 4);
    L->status = at; at += 256;
    L->workspace = at; at += up256(ws);
    L->total = at;
    return true;
}
}  // namespace

size_t fef_spec_verify_host_arena_bytes(int B, int K, int V, int64_t ld, fef_dtype dt) {
    ArenaLayout L;
    return arena_layout(B, K, V, ld, dt, &L) ? L.total : 0;
}

fef_status fef_spec_verify_host(const void* draft_logits, const void* target_logits, const int32_t* draft_tokens,
                                const int32_t* row_len, int B, int K, int V, int64_t ld, fef_dtype dt,
                                float temperature, uint64_t seed, uint32_t step, int32_t* accept_len,
                                int32_t* tokens, float* conf, int32_t* status_out, void* device_arena,
                                size_t device_arena_bytes, void* cuda_stream) {
    if (dt != FEF_F32 && dt != FEF_BF16) return FEF_ERR_DTYPE;
    if (!draft_logits || !target_logits || !draft_tokens || !accept_len || !tokens || !conf)
        return FEF_ERR_INVALID_ARG;
    ArenaLayout L;
    if (!arena_layout(B, K, V, ld, dt, &L)) {
        int dev;
        return cudaGetDevice(&dev) == cudaSuccess ? FEF_ERR_INVALID_ARG : FEF_ERR_CUDA;
    }
    if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255) || device_arena_bytes < L.total)
        return FEF_ERR_WORKSPACE;
    char* d = static_cast<char*>(device_arena);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t logits = static_cast<size_t>(B) * K * ld * (dt == FEF_F32 ? 4 : 2);
    const bool greedy = temperature == 0.0f;
    bool ok = true;
    if (!greedy) ok = ok && cudaMemcpyAsync(d + L.q, draft_logits, logits, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(d + L.p, target_logits, logits, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(d + L.tok, draft_tokens, static_cast<size_t>(B) * K * 4, cudaMemcpyHostToDevice,
                               stream) == cudaSuccess;
    if (row_len)
        ok = ok && cudaMemcpyAsync(d + L.row_len, row_len, static_cast<size_t>(B) * 4, cudaMemcpyHostToDevice,
                                   stream) == cudaSuccess;
    if (!ok) return FEF_ERR_CUDA;
    const fef_status st = fef_spec_verify(
        d + L.q, d + L.p, reinterpret_cast<const int32_t*>(d + L.tok),
        row_len ? reinterpret_cast<const int32_t*>(d + L.row_len) : nullptr, B, K, V, ld, dt, temperature, seed, step,
        reinterpret_cast<int32_t*>(d + L.accept_len), reinterpret_cast<int32_t*>(d + L.tokens),
        reinterpret_cast<float*>(d + L.conf), d + L.workspace, device_arena_bytes - L.workspace,
        reinterpret_cast<int32_t*>(d + L.status), cuda_stream);
    if (st != FEF_OK) return st;
    int32_t status_word = 0;
    ok = ok && cudaMemcpyAsync(accept_len, d + L.accept_len, static_cast<size_t>(B) * 4, cudaMemcpyDeviceToHost,
                               stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(tokens, d + L.tokens, static_cast<size_t>(B) * K * 4, cudaMemcpyDeviceToHost,
                               stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(conf, d + L.conf, static_cast<size_t>(B) * K * 4, cudaMemcpyDeviceToHost, stream) ==
                   cudaSuccess;
    ok = ok && cudaMemcpyAsync(&status_word, d + L.status, 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) return FEF_ERR_CUDA;
    if (status_out) *status_out = status_word;
    return FEF_OK;
}

// ---- variant for callers that cannot allocate device memory
//
// Scratch for fef_spec_verify_static.  It is part of the library image: every GPU that loads
// the library carries these FEF_STATIC_SCRATCH_BYTES until the process exits.  In host code
// the name below is only a handle for the runtime (not a device address); the address the
// kernels get comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[FEF_STATIC_SCRATCH_BYTES];
static void* g_static_scratch_address[64];  // per device, filled on the first call there

fef_status fef_spec_verify_static(const void* draft_logits, const void* target_logits, const int32_t* draft_tokens,
                                  const int32_t* row_len, int B, int K, int V, int64_t ld, fef_dtype dt,
                                  float temperature, uint64_t seed, uint32_t step, int32_t* accept_len,
                                  int32_t* tokens, float* conf, int32_t* device_status, void* cuda_stream) {
    if (dt != FEF_F32 && dt != FEF_BF16) return FEF_ERR_DTYPE;
    if (B < 1 || B > FEF_MAX_B || K < 1 || K > FEF_MAX_K || V < 1 || ld < V) return FEF_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FEF_ERR_CUDA;
    const size_t need = fef_spec_verify_workspace_bytes(B, K, V, dt);
    if (need == 0) return FEF_ERR_INVALID_ARG;
    if (need > FEF_STATIC_SCRATCH_BYTES) return FEF_ERR_TOO_LARGE;
    void* scratch = g_static_scratch_address[dev];
    if (!scratch) {
        // set-up, once per device, with that device current: ask the runtime where the array lives
        if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) return FEF_ERR_CUDA;
        g_static_scratch_address[dev] = scratch;
    }
    // The array keeps what the previous call left.  fef_spec_verify clears the part that must
    // start at zero (the streaming kernel's claim counter) on the stream before its kernels;
    // every other value is written before it is read (the scan kernel rewrites every window's
    // task, arrival counter included), so leftovers of earlier calls are never used.
    return fef_spec_verify(draft_logits, target_logits, draft_tokens, row_len, B, K, V, ld, dt, temperature, seed,
                           step, accept_len, tokens, conf, scratch, FEF_STATIC_SCRATCH_BYTES, device_status,
                           cuda_stream);
}

}  // extern "C"

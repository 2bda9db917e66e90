// Device helpers shared by the kernels of the verification library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fef.h"

namespace fef {

// ------------------------------------------------------------------ sizes ----
constexpr int kConsumerWarps = 16;                      // warps that do arithmetic in the streaming kernel
constexpr int kProducerWarp = kConsumerWarps;           // one thread of it feeds the ring
constexpr int kStreamThreads = (kConsumerWarps + 1) * 32;
constexpr int kVecPerThread = 4;                        // 16-byte vectors per thread per chunk
constexpr int kChunkBytes = kConsumerWarps * 32 * 16 * kVecPerThread;  // 32 KiB: what the consumers take in one go
constexpr int kHalves = 2;                              // chunks per tile: one barrier wait and one release per 64 KiB
constexpr int kTileBytes = kChunkBytes * kHalves;       // 64 KiB
constexpr int kStages = 3;                              // ring depth: 192 KiB in flight per SM
constexpr unsigned long long kWaitLimitNs = 1000000000ull;  // a wait inside a kernel gives up after this long (1 s)
constexpr int kSpinRounds = 1 << 24;                    // ... or after this many rounds of 64 polls, whichever comes first
constexpr int kSlotSets = 8;                            // in-CTA combine buffers (a warp leads by < 8 flushes)

constexpr float kNoReference = -3.0e38f;                // "no reference yet" for the running softmax
constexpr float kRescaleAbove = 1.152921504606847e18f;  // 2^60: a vector sum above this re-references

// One partial result of the streaming kernel: one claim's share of one row.
//   ref    reference exponent (log2 domain) the sum is relative to
//   sum    sum_v 2^(l_v * c - ref) over the claim's elements (NaN when the data is bad)
//   best   largest logit seen (greedy mode only)
//   index  vocabulary id of `best`, lowest on ties (greedy mode only)
struct __align__(16) Partial {
    float ref;
    float sum;
    float best;
    int index;
};

// Per-window hand-over from the scan kernel to the residual kernel.
// (The single-GPU call decides the rejected position inside its last kernel and uses only the
// arrival counter; the vocabulary-parallel steps hand the whole record from one call to the next.)
struct __align__(16) ResidualTask {
    int pos;            // rejected position a, or -1 when the window has no residual draw
    unsigned arrivals;  // CTAs of the residual draw that have finished their share of this window
    double kp;          // log2 normaliser of the target law at a: pi(x) = 2^(l_x * c - kp)
    double kq;          // same for the draft law
};

// Shared by all CTAs of the streaming kernel (cleared by begin_call_kernel, the call's first kernel).
struct __align__(16) Control {
    unsigned long long next_claim;  // next streaming claim to hand out
    int aborted;                    // a bounded wait ran out: the partials are incomplete, no window is decided
};

// Vocabulary-parallel verification: what one rank reports for a rejected window after its
// share of the residual draw.
struct __align__(16) VpCandidate {
    double score;  // exact Gumbel score ln r - ln(-ln u) of the rank's best id, -inf if its slice has no r > 0
    float lp;      // target logit of `index`
    int index;     // global vocabulary id: the best id, or (score = -inf) the slice's arg-max of the target logits
};

struct __align__(8) Candidate {
    float w;  // r_x / (-ln u_x) in binary32, <= 0 when empty
    int x;
};

// ------------------------------------------------------------ small maths ----
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}


// Philox4x32-10 (Salmon et al. 2011): returns the four output words.
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint2 key) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = static_cast<uint64_t>(M0) * ctr.x;  // one wide multiply gives both halves
        const uint64_t p1 = static_cast<uint64_t>(M1) * ctr.z;
        ctr = make_uint4(static_cast<uint32_t>(p1 >> 32) ^ ctr.y ^ key.x, static_cast<uint32_t>(p1),
                         static_cast<uint32_t>(p0 >> 32) ^ ctr.w ^ key.y, static_cast<uint32_t>(p0));
        key.x += W0;
        key.y += W1;
    }
    return ctr;
}

// The same generator for many counters that differ in their first word only (one batch row,
// one window position, one call).  The ten round keys come precomputed (kernel-parameter
// constants, so they cost no instruction), and the parts of rounds one and two that depend on
// the fixed words alone are worked out once per row.
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
};
inline PhiloxKeys philox_round_keys(uint64_t seed) {
    PhiloxKeys k;
    uint32_t a = static_cast<uint32_t>(seed), b = static_cast<uint32_t>(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = a;
        k.k1[r] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return k;
}
struct PhiloxRow {
    uint32_t s1, a1k, c2, d3;
    __device__ __forceinline__ void prepare(const PhiloxKeys& K, uint32_t c1, uint32_t c2_, uint32_t c3) {
        constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
        const uint64_t p = static_cast<uint64_t>(M1) * c2_;
        const uint32_t a0 = static_cast<uint32_t>(p >> 32) ^ c1 ^ K.k0[0];   // word 0 after round one
        s1 = c3 ^ K.k1[0];
        a1k = static_cast<uint32_t>(p) ^ K.k0[1];                            // word 1 after round one, keyed
        const uint64_t q = static_cast<uint64_t>(M0) * a0;
        c2 = static_cast<uint32_t>(q >> 32) ^ K.k1[1];
        d3 = static_cast<uint32_t>(q) ^ K.k1[2];                             // word 3 after round two, keyed
    }
    __device__ __forceinline__ uint4 draw(const PhiloxKeys& K, uint32_t c0) const {
        constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
        uint64_t p0 = static_cast<uint64_t>(M0) * c0;                         // round one
        const uint32_t v2 = static_cast<uint32_t>(p0 >> 32) ^ s1, v3 = static_cast<uint32_t>(p0);
        uint64_t p1 = static_cast<uint64_t>(M1) * v2;                         // round two
        const uint32_t w0 = static_cast<uint32_t>(p1 >> 32) ^ a1k, w1 = static_cast<uint32_t>(p1), w2 = v3 ^ c2;
        p0 = static_cast<uint64_t>(M0) * w0;                                  // round three
        p1 = static_cast<uint64_t>(M1) * w2;
        uint4 ctr = make_uint4(static_cast<uint32_t>(p1 >> 32) ^ w1 ^ K.k0[2], static_cast<uint32_t>(p1),
                               static_cast<uint32_t>(p0 >> 32) ^ d3, static_cast<uint32_t>(p0));
#pragma unroll
        for (int r = 3; r < 10; ++r) {
            p0 = static_cast<uint64_t>(M0) * ctr.x;
            p1 = static_cast<uint64_t>(M1) * ctr.z;
            ctr = make_uint4(static_cast<uint32_t>(p1 >> 32) ^ ctr.y ^ K.k0[r], static_cast<uint32_t>(p1),
                             static_cast<uint32_t>(p0 >> 32) ^ ctr.w ^ K.k1[r], static_cast<uint32_t>(p0));
        }
        return ctr;
    }
};

// 23 random bits centred in their bin: u in (0, 1), exact in binary32.
__device__ __forceinline__ float uniform_from_word(uint32_t r) {
    return (static_cast<float>(r >> 9) + 0.5f) * (1.0f / 8388608.0f);
}

constexpr uint32_t kStreamAccept = 0u;
constexpr uint32_t kStreamResidual = 1u;

// ------------------------------------------------------ loads and unpacking ----
template <int DT>
struct Elem;
template <>
struct Elem<FEF_F32> {
    static constexpr int kBytes = 4;
    static constexpr int kPerVec = 4;
    static constexpr bool kSplitScale = true;   // c = c_hi + c_lo, two fused multiply-adds
};
template <>
struct Elem<FEF_BF16> {
    static constexpr int kBytes = 2;
    static constexpr int kPerVec = 8;
    static constexpr bool kSplitScale = false;  // c = c_hi alone (c_lo is 0)
};

// 2^(l * c - ref).  With the split scale c = c_hi + c_lo and c_lo > 0, so l = -inf stays -inf.
template <int DT>
__device__ __forceinline__ float exp2_scaled(float l, float c_hi, float c_lo, float ref) {
    float x = fmaf(l, c_hi, -ref);
    if constexpr (Elem<DT>::kSplitScale) x = fmaf(l, c_lo, x);
    return ex2_approx(x);
}

template <int DT>
__device__ __forceinline__ void unpack(const uint4& w, float (&l)[Elem<DT>::kPerVec]) {
    if constexpr (DT == FEF_F32) {
        l[0] = __uint_as_float(w.x);
        l[1] = __uint_as_float(w.y);
        l[2] = __uint_as_float(w.z);
        l[3] = __uint_as_float(w.w);
    } else {
        // a bfloat16 is the upper half of a binary32
        l[0] = __uint_as_float(w.x << 16);
        l[1] = __uint_as_float(w.x & 0xFFFF0000u);
        l[2] = __uint_as_float(w.y << 16);
        l[3] = __uint_as_float(w.y & 0xFFFF0000u);
        l[4] = __uint_as_float(w.z << 16);
        l[5] = __uint_as_float(w.z & 0xFFFF0000u);
        l[6] = __uint_as_float(w.w << 16);
        l[7] = __uint_as_float(w.w & 0xFFFF0000u);
    }
}

template <int DT>
__device__ __forceinline__ float load_logit(const void* row, int64_t v) {
    if constexpr (DT == FEF_F32) {
        return __ldg(static_cast<const float*>(row) + v);
    } else {
        const uint32_t h = __ldg(static_cast<const unsigned short*>(row) + v);
        return __uint_as_float(h << 16);
    }
}

__device__ __forceinline__ uint4 ld_global_nc_v4(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// --------------------------------------------------- mbarrier and bulk copy ----
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when `limit_ns` of wall time have passed (the poll count is a second bound,
// should the timer not advance) or another thread already gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                  unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long start = globaltimer_ns();
    for (int round = 0; round < kSpinRounds; ++round) {
        for (int spin = 0; spin < 64; ++spin)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (globaltimer_ns() - start > limit_ns) return false;
    }
    return false;
}
// 1-D bulk copy global -> shared, completion counted in bytes on `bar`.
// dst, src and bytes must be multiples of 16.
// The logits are read once: they are marked "evict first" in L2, so that they do not push out
// what the following kernels and calls reuse (`policy` from l2_evict_first_policy()).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// Ordered 64-bit key for "largest w, then lowest x".
__device__ __forceinline__ bool better(float w, int x, float w2, int x2) {
    return w > w2 || (w == w2 && x < x2);
}

}  // namespace fef

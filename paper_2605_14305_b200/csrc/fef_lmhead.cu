// fef_lmhead_verify: verification straight from hidden states.  The draft and target laws of
// Section 3.2 are model outputs, logits = hidden state x output-layer weight; here that product
// runs on the tensor cores (tcgen05.mma, accumulators in tensor memory, operands brought in by
// TMA) and its epilogue reduces every accumulator tile to the softmax partials the verification
// needs, so the [B*K, V] logits never reach HBM:
//   lmhead_gemm_kernel<kStats>   logits tile by tile -> per (row, vocabulary chunk) the pair
//                                (reference exponent, sum of 2^(l c - ref)) and the logit at the draft token;
//   lmhead_accept_kernel         one CTA per window: normalisers in double precision, acceptance tests,
//                                first rejection, accepted tokens and confidences (Algorithm 2's loop);
//                                gathers the hidden states of the rejected positions;
//   lmhead_gemm_kernel<kStore>   the logits of the rejected positions only (2 B rows), in binary32;
//   lmhead_residual_kernel       the residual draw on those rows (fef_residual.cuh).
// The logits are the binary32 accumulations of the bfloat16 products as the tensor cores deliver
// them; they are never rounded to bfloat16.
//
// GEMM kernel: one CTA per SM, persistent over work items (128 rows x a run of 256-column tiles).
// Warp 0: TMA producer (one thread) into a 4-stage ring of 128x64 (A) and 256x64 (B) bfloat16 tiles
// in the 128-byte-swizzled K-major layout.  Warp 1: issues the MMAs (one thread; 128x256x16 per
// instruction, four per stage) into one of two 256-column accumulators in tensor memory and
// commits them to mbarriers.  Warps 2-5: epilogue, one accumulator row per thread
// (tcgen05.ld 32 columns at a time), overlapping the next tile's MMAs.  Every wait is bounded.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"
#include "fef_device_math.cuh"
#include "fef_verify_params.cuh"
#include "fef_residual.cuh"

namespace fef {
namespace lm {

constexpr int kBM = 128, kBN = 256, kBK = 64;  // CTA tile; kBK bfloat16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;                     // K of one tcgen05.mma (kind::f16)
constexpr int kGemmStages = 4;
constexpr int kABytes = kBM * kBK * 2;         // 16 KiB
constexpr int kBBytes = kBN * kBK * 2;         // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTmemCols = 512;                 // two accumulators of kBN columns
constexpr int kGemmThreads = 192;              // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kEpilogueWarps = 4;
constexpr unsigned long long kGemmWaitNs = 1000000000ull;

enum : int { kStats = 0, kStore = 1 };

struct __align__(8) ChunkPartial {
    float ref;  // reference exponent (log2 domain)
    float sum;  // sum of 2^(l c - ref) over the chunk's columns (NaN: bad data)
};

struct GemmParams {
    int m_tiles;            // row tiles of both operand matrices together
    int m_tiles_first;      // row tiles of the first matrix (the second follows)
    int n_tiles;            // 256-column tiles of the vocabulary
    int k_blocks;           // 64-deep blocks of the hidden width
    int tiles_per_chunk;    // column tiles one work item covers
    int chunks;             // ceil(n_tiles / tiles_per_chunk)
    int rows;               // valid rows per matrix
    int V;
    float c;                // log2(e) / T
    const int32_t* tokens;  // kStats: [rows] draft token of each row (of both matrices), or null
    const int32_t* row_len; // kStats: [B] or null
    int K;                  // window length (row = b * K + i)
    ChunkPartial* partials; // kStats: [2][rows][chunks]
    float* logit_at_token;  // kStats: [2][rows]
    float* logits_out;      // kStore: [rows of both matrices][ldo]
    int64_t ldo;
    int32_t* status;
};

struct GemmShared {
    uint64_t full[kGemmStages];
    uint64_t empty[kGemmStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t drained;
    uint32_t tmem_base;
    int abort_flag;
};
constexpr size_t kGemmSmemBytes = static_cast<size_t>(kGemmStages) * kStageBytes + sizeof(GemmShared) + 1024;

// ---- PTX wrappers (sm_100a)
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 256 x 16, bfloat16 inputs, binary32 accumulation.
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t"
        "}\n" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// 32 consecutive columns of this thread's accumulator row.
__device__ __forceinline__ void tmem_load32(uint32_t addr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major bfloat16 tile in the 128-byte-swizzled layout (rows of
// 128 bytes, groups of eight rows 1024 bytes apart): start address, stride between row groups, layout
// type, descriptor version of this architecture.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu);   // start address (16-byte units)
    d |= static_cast<uint64_t>(1u) << 16;                     // leading byte offset (not used by swizzled K-major)
    d |= static_cast<uint64_t>(1024u >> 4) << 32;             // stride byte offset: eight rows
    d |= static_cast<uint64_t>(1u) << 46;                     // descriptor version
    d |= static_cast<uint64_t>(2u) << 61;                     // 128-byte swizzle
    return d;
}
// Instruction descriptor: binary32 accumulator, bfloat16 A and B, both K-major, N = 256, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kBN >> 3) << 17) | ((kBM >> 4) << 24);

template <int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
lmhead_gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                   const __grid_constant__ CUtensorMap map_b, const __grid_constant__ GemmParams P) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    GemmShared& sh = *reinterpret_cast<GemmShared*>(smem + kGemmStages * kStageBytes);
    volatile int* abort_flag = &sh.abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemmStages; ++s) {
            mbar_init(sh.full + s, 1);
            mbar_init(sh.empty + s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(sh.tmem_full + a, 1);
            mbar_init(sh.tmem_empty + a, kEpilogueWarps);
        }
        mbar_init(&sh.drained, 1);
        sh.abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(&sh.tmem_base, kTmemCols);  // (one CTA per SM: the columns are always free)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&sh.tmem_base);
    cudaGridDependencySynchronize();

    const int items = P.m_tiles * P.chunks;
    int issued = 0;  // stages put in flight (producer thread)

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < items; item += gridDim.x) {
                const int chunk = item / P.m_tiles, m = item - chunk * P.m_tiles;
                const CUtensorMap* map_a = m < P.m_tiles_first ? &map_a0 : &map_a1;
                const int row0 = (m < P.m_tiles_first ? m : m - P.m_tiles_first) * kBM;
                const int n_begin = chunk * P.tiles_per_chunk, n_end = min(n_begin + P.tiles_per_chunk, P.n_tiles);
                for (int n = n_begin; ok && n < n_end; ++n)
                    for (int kb = 0; kb < P.k_blocks; ++kb) {
                        if (!mbar_wait_bounded(sh.empty + stage, phase ^ 1u, abort_flag, kGemmWaitNs)) {
                            *abort_flag = 1;
                            report(P.status, FEF_ERR_TIMEOUT);
                            ok = false;
                            break;
                        }
                        unsigned char* a_dst = smem + stage * kStageBytes;
                        mbar_arrive_expect_tx(sh.full + stage, kStageBytes);
                        tma_load_2d(a_dst, map_a, kb * kBK, row0, sh.full + stage);
                        tma_load_2d(a_dst + kABytes, &map_b, kb * kBK, n * kBN, sh.full + stage);
                        ++issued;
                        if (++stage == kGemmStages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            unsigned uses[2] = {0u, 0u};
            unsigned tile = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < items; item += gridDim.x) {
                const int chunk = item / P.m_tiles;
                const int n_begin = chunk * P.tiles_per_chunk, n_end = min(n_begin + P.tiles_per_chunk, P.n_tiles);
                for (int n = n_begin; ok && n < n_end; ++n, ++tile) {
                    const int acc = tile & 1;
                    // the epilogue must have drained this accumulator (passes at once on its first use)
                    if (!mbar_wait_bounded(sh.tmem_empty + acc, (uses[acc] & 1u) ^ 1u, abort_flag, kGemmWaitNs)) {
                        *abort_flag = 1;
                        report(P.status, FEF_ERR_TIMEOUT);
                        ok = false;
                        break;
                    }
                    ++uses[acc];
                    tc_fence_after();
                    const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(acc * kBN);
                    for (int kb = 0; kb < P.k_blocks; ++kb) {
                        if (!mbar_wait_bounded(sh.full + stage, phase, abort_flag, kGemmWaitNs)) {
                            *abort_flag = 1;
                            report(P.status, FEF_ERR_TIMEOUT);
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t a_addr = smem_u32(smem + stage * kStageBytes);
                        const uint64_t desc_a = smem_desc_sw128(a_addr), desc_b = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kBK / kUmmaK; ++k)  // 32 bytes further along K inside the swizzle row
                            tc_mma(tmem_d, desc_a + static_cast<uint64_t>(2 * k), desc_b + static_cast<uint64_t>(2 * k),
                                   kInstrDesc, (kb | k) != 0 ? 1u : 0u);
                        tc_commit(sh.empty + stage);  // arrives when these MMAs have read the stage
                        if (++stage == kGemmStages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (ok) tc_commit(sh.tmem_full + acc);  // arrives when the tile's accumulator is complete
                }
            }
            // everything issued has finished before the tensor memory goes back
            tc_commit(&sh.drained);
            mbar_wait_bounded(&sh.drained, 0u, abort_flag, kGemmWaitNs);
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int quarter = warp & 3;                 // the tensor-memory lanes this warp may read
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        unsigned uses[2] = {0u, 0u};
        unsigned tile = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < items; item += gridDim.x) {
            const int chunk = item / P.m_tiles, m = item - chunk * P.m_tiles;
            const int which = m < P.m_tiles_first ? 0 : 1;
            const int row = (which ? m - P.m_tiles_first : m) * kBM + row_in_tile;
            const bool valid = row < P.rows;
            const int n_begin = chunk * P.tiles_per_chunk, n_end = min(n_begin + P.tiles_per_chunk, P.n_tiles);
            float ref = -INFINITY, sum = 0.f, lx = 0.f;
            bool have_lx = false;
            int tok = -1;
            if (MODE == kStats && valid && P.tokens) {
                const int b = row / P.K, i = row - b * P.K;
                const int nb = P.row_len ? __ldg(P.row_len + b) : P.K;
                if (i < nb) tok = __ldg(P.tokens + row);
            }
            for (int n = n_begin; ok && n < n_end; ++n, ++tile) {
                const int acc = tile & 1;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(sh.tmem_full + acc, uses[acc] & 1u, abort_flag, kGemmWaitNs))) {
                    *abort_flag = 1;
                    report(P.status, FEF_ERR_TIMEOUT);
                    ok = false;
                    break;
                }
                ++uses[acc];
                tc_fence_after();
#pragma unroll 1
                for (int c8 = 0; c8 < kBN / 32; ++c8) {
                    const int col0 = n * kBN + c8 * 32;
                    if (col0 >= P.V) break;  // (uniform over the warp)
                    float v[32];
                    tmem_load32(lane_addr + static_cast<uint32_t>(acc * kBN + c8 * 32), v);
                    if (col0 + 32 > P.V) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col0 + j >= P.V) v[j] = -INFINITY;
                    }
                    if constexpr (MODE == kStats) {
                        float cm = v[0];
#pragma unroll
                        for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
                        const float x = cm * P.c;
                        if (x > ref) {  // (NaN compares false and poisons the sum below)
                            sum *= ex2_approx(ref - x);
                            ref = x;
                        }
                        float s0 = 0.f, s1 = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            s0 += ex2_approx(fmaf(v[j], P.c, -ref));
                            s1 += ex2_approx(fmaf(v[j + 1], P.c, -ref));
                        }
                        sum += s0 + s1;
                        if (static_cast<unsigned>(tok - col0) < 32u) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (tok - col0 == j) lx = v[j];
                            have_lx = true;
                        }
                    } else {
                        if (valid) {
                            float* out = P.logits_out + (static_cast<int64_t>(which) * P.rows + row) * P.ldo + col0;
                            if (col0 + 32 <= P.V) {
#pragma unroll
                                for (int j = 0; j < 32; j += 4)
                                    *reinterpret_cast<float4*>(out + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (col0 + j < P.V) out[j] = v[j];
                            }
                        }
                    }
                }
                // the accumulator may be overwritten
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(sh.tmem_empty + acc);
            }
            if (MODE == kStats && ok && valid) {
                ChunkPartial rec;
                rec.ref = ref;
                rec.sum = sum;
                P.partials[(static_cast<int64_t>(which) * P.rows + row) * P.chunks + chunk] = rec;
                if (have_lx) P.logit_at_token[static_cast<int64_t>(which) * P.rows + row] = lx;
            }
        }
    }

    // ---- teardown: copies still in flight after an abort get a bounded chance to land; then the
    //      tensor memory goes back
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        const int first = issued > kGemmStages ? issued - kGemmStages : 0;
        for (int k = first; k < issued; ++k) {
            volatile int never = 0;
            mbar_wait_bounded(sh.full + (k % kGemmStages), static_cast<uint32_t>((k / kGemmStages) & 1), &never, kGemmWaitNs);
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ================================================================ accept ====
// Acceptance tests of one window from the chunk partials (Algorithm 2's loop over the window's
// positions): one CTA per window, a warp per position folding its partials in double precision.
struct AcceptParams {
    int B, K, V, chunks, rows, d;
    float c;
    const ChunkPartial* partials;   // [2][rows][chunks]: target, then draft
    const float* logit_at_token;    // [2][rows]
    const int32_t* tokens;
    const int32_t* row_len;
    const uint16_t* target_hidden;  // [rows][d]
    const uint16_t* draft_hidden;
    uint16_t* gathered;             // [2 * B][d]: target rows of the rejected positions, then draft rows
    uint64_t seed;
    uint32_t step;
    int32_t* accept_len;
    int32_t* out_tokens;
    float* conf;
    ResidualTask* tasks;
    int32_t* status;
};

constexpr int kAcceptThreads = 256;

// (reference, sum) of one law at one row from its chunk partials; false on bad data.
__device__ bool fold_chunks(const ChunkPartial* rec, int chunks, int lane, double* k_out) {
    double m = -INFINITY, s = 0.0;
    int bad = 0;
    for (int r = lane; r < chunks; r += 32) {
        const ChunkPartial p = rec[r];
        if (!(p.sum >= 0.f) || p.sum == INFINITY) bad = 1;
        if (p.sum > 0.f) {
            const double pm = p.ref, ps = p.sum;
            if (pm > m) {
                s = m > -INFINITY ? s * exp2(m - pm) + ps : ps;
                m = pm;
            } else {
                s += pm == m ? ps : ps * exp2(pm - m);
            }
        }
    }
    const double M = warp_max(m);
    bad = __any_sync(0xFFFFFFFFu, bad);
    const double S = warp_sum(m > -INFINITY ? s * exp2(m - M) : 0.0);
    if (bad || !(S > 0.0) || !(S < INFINITY)) return false;
    *k_out = M + log2(S);
    return true;
}

__global__ void __launch_bounds__(kAcceptThreads) lmhead_accept_kernel(const __grid_constant__ AcceptParams P) {
    cudaGridDependencySynchronize();
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = P.row_len ? min(max(__ldg(P.row_len + b), 0), P.K) : P.K;
    const double c = static_cast<double>(P.c);
    __shared__ double s_kp[FEF_MAX_K], s_kq[FEF_MAX_K];
    __shared__ float s_conf[FEF_MAX_K];
    __shared__ int s_accept[FEF_MAX_K], s_err[FEF_MAX_K];
    for (int i = warp; i < n; i += kAcceptThreads / 32) {
        const int64_t row = static_cast<int64_t>(b) * P.K + i;
        double kp = 0.0, kq = 0.0;
        const bool okp = fold_chunks(P.partials + row * P.chunks, P.chunks, lane, &kp);
        const bool okq = fold_chunks(P.partials + (static_cast<int64_t>(P.rows) + row) * P.chunks, P.chunks, lane, &kq);
        if (lane == 0) {
            const int x = __ldg(P.tokens + row);
            int err = 0, accept = 0;
            float conf = -1.f;
            if (x < 0 || x >= P.V) {
                err = FEF_ERR_TOKEN_RANGE;
            } else if (!okp || !okq) {
                err = FEF_ERR_NONFINITE;
            } else {
                const double lpx = P.logit_at_token[row], lqx = P.logit_at_token[P.rows + row];
                const double l2pi = lpx * c - kp;
                conf = static_cast<float>(exp2(l2pi));
                const double ratio = exp2(l2pi - (lqx * c - kq));
                const uint4 rnd = philox4x32_10(
                    make_uint4(kStreamAccept << 30, static_cast<uint32_t>(b), static_cast<uint32_t>(i), P.step),
                    make_uint2(static_cast<uint32_t>(P.seed), static_cast<uint32_t>(P.seed >> 32)));
                accept = static_cast<double>(uniform_from_word(rnd.x)) <= fmin(1.0, ratio);
            }
            s_err[i] = err;
            s_accept[i] = accept;
            s_conf[i] = conf;
            s_kp[i] = kp;
            s_kq[i] = kq;
        }
    }
    __syncthreads();
    int err = 0, a = n;
    for (int i = 0; i < n; ++i) err = max(err, s_err[i]);
    for (int i = n - 1; i >= 0; --i)
        if (!s_accept[i]) a = i;
    for (int i = threadIdx.x; i < P.K; i += kAcceptThreads) {
        const int64_t row = static_cast<int64_t>(b) * P.K + i;
        const bool keep = !err && i < a;
        P.out_tokens[row] = keep ? __ldg(P.tokens + row) : -1;
        P.conf[row] = keep ? s_conf[i] : -1.f;
    }
    const bool rejected = !err && a < n;
    if (threadIdx.x == 0) {
        P.accept_len[b] = err ? -1 : a;
        if (err) report(P.status, err);
        ResidualTask task;
        task.pos = rejected ? a : -1;
        task.arrivals = 0u;
        task.kp = rejected ? s_kp[a] : 0.0;
        task.kq = rejected ? s_kq[a] : 0.0;
        P.tasks[b] = task;
    }
    // the rejected position's two hidden states, side by side for the second product (zeros when
    // nothing was rejected, so that its rows stay finite)
    const int64_t src = (static_cast<int64_t>(b) * P.K + (rejected ? a : 0)) * P.d;
    for (int k = threadIdx.x; k < P.d; k += kAcceptThreads) {
        P.gathered[static_cast<int64_t>(b) * P.d + k] = rejected ? P.target_hidden[src + k] : uint16_t(0);
        P.gathered[(static_cast<int64_t>(P.B) + b) * P.d + k] = rejected ? P.draft_hidden[src + k] : uint16_t(0);
    }
}

// ============================================================== residual ====
// The residual draw on the binary32 logits of the rejected positions ([2 B][ldo]: target rows, then
// draft rows), shared by `parts` CTAs per window.
__global__ void __launch_bounds__(kResidualThreads, kResidualCtasPerSm)
lmhead_residual_kernel(const __grid_constant__ VerifyParams P, const float* __restrict__ logits, int64_t ldo) {
    __shared__ ResidualShared sh;
    cudaGridDependencySynchronize();
    const int b = blockIdx.y;
    const ResidualTask task = P.tasks[b];
    if (task.pos < 0) return;  // uniform over the CTA
    if (threadIdx.x == 0) sh.floor_bits = sh.best3[0] = sh.best3[1] = sh.best3[2] = 0u;
    __syncthreads();
    const char* prow = reinterpret_cast<const char*>(logits + static_cast<int64_t>(b) * ldo);
    const char* qrow = reinterpret_cast<const char*>(logits + (static_cast<int64_t>(P.geo.B) + b) * ldo);
    residual_draw<FEF_F32, false, false>(P, b, task.pos, task.kp, task.kq, prow, qrow,
                                         static_cast<int64_t>(b) * P.geo.K + task.pos, blockIdx.x, gridDim.x, sh);
}

// ================================================================== host ====
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map of a row-major bfloat16 matrix [rows][d] with boxes of box_rows x 64 elements, 128-byte swizzle.
static bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t d, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 2};
    const cuuint32_t box[2] = {kBK, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int g_lm_sms[64];
static bool g_lm_attr[64][2];

static int lm_sm_count(int* dev_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (g_lm_sms[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        g_lm_sms[dev] = n;
    }
    *dev_out = dev;
    return g_lm_sms[dev];
}

template <typename... Args>
static cudaError_t launch_pdl(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
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

// One product: rows of `a0` (and, if given, of `a1`) times `weight`^T, epilogue MODE.
template <int MODE>
static cudaError_t launch_gemm(const void* a0, const void* a1, int rows, const void* weight, int V, int d, GemmParams P,
                               int dev, int sms, cudaStream_t stream) {
    CUtensorMap ma0, ma1, mb;
    if (!make_map(&ma0, a0, rows, d, kBM) || !make_map(&ma1, a1 ? a1 : a0, rows, d, kBM) || !make_map(&mb, weight, V, d, kBN))
        return cudaErrorInvalidValue;
    if (!g_lm_attr[dev][MODE]) {
        const cudaError_t e = cudaFuncSetAttribute(lmhead_gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   static_cast<int>(kGemmSmemBytes));
        if (e != cudaSuccess) return e;
        g_lm_attr[dev][MODE] = true;
    }
    const int per = (rows + kBM - 1) / kBM;
    P.m_tiles_first = per;
    P.m_tiles = a1 ? 2 * per : per;
    P.n_tiles = (V + kBN - 1) / kBN;
    P.k_blocks = (d + kBK - 1) / kBK;
    P.rows = rows;
    P.V = V;
    if (MODE == kStore) P.tiles_per_chunk = 1;
    P.chunks = (P.n_tiles + P.tiles_per_chunk - 1) / P.tiles_per_chunk;
    const int items = P.m_tiles * P.chunks;
    const int grid = items < sms ? items : sms;
    return launch_pdl(lmhead_gemm_kernel<MODE>, dim3(grid), dim3(kGemmThreads), kGemmSmemBytes, stream, ma0, ma1, mb, P);
}

static int stats_tiles_per_chunk(int rows, int V, int sms) {
    const int m_tiles = 2 * ((rows + kBM - 1) / kBM), n_tiles = (V + kBN - 1) / kBN;
    int tpc = static_cast<int>(static_cast<int64_t>(m_tiles) * n_tiles / (static_cast<int64_t>(sms) * 16));
    if (tpc < 1) tpc = 1;
    if (tpc > 16) tpc = 16;
    return tpc;
}

struct LmLayout {
    size_t partials, lx, tasks, gathered, logits, candidates, total;
    int chunks;
    int64_t ldo;
};
static size_t lm_round(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }
static LmLayout lm_layout(int B, int K, int V, int d, int sms) {
    LmLayout L;
    const int rows = B * K;
    const int tpc = stats_tiles_per_chunk(rows, V, sms);
    const int n_tiles = (V + kBN - 1) / kBN;
    L.chunks = (n_tiles + tpc - 1) / tpc;
    L.ldo = (static_cast<int64_t>(V) + 3) / 4 * 4;
    size_t at = 0;
    L.partials = at; at += lm_round(static_cast<size_t>(2) * rows * L.chunks * sizeof(ChunkPartial));
    L.lx = at; at += lm_round(static_cast<size_t>(2) * rows * sizeof(float));
    L.tasks = at; at += lm_round(static_cast<size_t>(B) * sizeof(ResidualTask));
    L.gathered = at; at += lm_round(static_cast<size_t>(2) * B * d * 2);
    L.logits = at; at += lm_round(static_cast<size_t>(2) * B * L.ldo * sizeof(float));
    L.candidates = at; at += lm_round(static_cast<size_t>(B) * kMaxResidualCtas * kCandidatesPerCta * sizeof(Candidate));
    L.total = at;
    return L;
}

static bool lm_sizes_ok(int B, int K, int V, int d) {
    return B >= 1 && B <= FEF_MAX_B && K >= 1 && K <= FEF_MAX_K && V >= 1 && d >= 8 && (d % 8) == 0 &&
           static_cast<int64_t>(B) * K < (1 << 24) && static_cast<int64_t>(V) * 4 <= (1ll << 30);
}

}  // namespace lm
}  // namespace fef

extern "C" {

size_t fef_lmhead_verify_workspace_bytes(int B, int K, int V, int d) {
    using namespace fef::lm;
    int dev = 0;
    const int sms = lm_sm_count(&dev);
    if (sms < 1 || !lm_sizes_ok(B, K, V, d)) return 0;
    return lm_layout(B, K, V, d, sms).total;
}

fef_status fef_lmhead_logits(const void* hidden, const void* weight, int rows, int V, int d, float* logits, int64_t ldo,
                             int32_t* device_status, void* cuda_stream) {
    using namespace fef;
    using namespace fef::lm;
    if (!hidden || !weight || !logits) return FEF_ERR_INVALID_ARG;
    if (rows < 1 || V < 1 || d < 8 || (d % 8) || ldo < V || (ldo % 4)) return FEF_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15) || (reinterpret_cast<uintptr_t>(weight) & 15) ||
        (reinterpret_cast<uintptr_t>(logits) & 15))
        return FEF_ERR_ALIGNMENT;
    int dev = 0;
    const int sms = lm_sm_count(&dev);
    if (sms < 1) return FEF_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (device_status && cudaMemsetAsync(device_status, 0, sizeof(int32_t), stream) != cudaSuccess) return FEF_ERR_CUDA;
    GemmParams P = {};
    P.c = 1.f;
    P.K = 1;
    P.logits_out = logits;
    P.ldo = ldo;
    P.status = device_status;
    const cudaError_t e = launch_gemm<kStore>(hidden, nullptr, rows, weight, V, d, P, dev, sms, stream);
    return e == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_lmhead_verify(const void* draft_hidden, const void* target_hidden, const void* weight,
                             const int32_t* draft_tokens, const int32_t* row_len, int B, int K, int V, int d,
                             float temperature, uint64_t seed, uint32_t step, int32_t* accept_len, int32_t* tokens,
                             float* conf, void* workspace, size_t workspace_bytes, int32_t* device_status,
                             void* cuda_stream) {
    using namespace fef;
    using namespace fef::lm;
    if (!draft_hidden || !target_hidden || !weight || !draft_tokens || !accept_len || !tokens || !conf)
        return FEF_ERR_INVALID_ARG;
    if (!lm_sizes_ok(B, K, V, d)) return FEF_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || isinf(temperature)) return FEF_ERR_INVALID_ARG;  // sampling mode
    if ((reinterpret_cast<uintptr_t>(draft_hidden) & 15) || (reinterpret_cast<uintptr_t>(target_hidden) & 15) ||
        (reinterpret_cast<uintptr_t>(weight) & 15))
        return FEF_ERR_ALIGNMENT;
    int dev = 0;
    const int sms = lm_sm_count(&dev);
    if (sms < 1) return FEF_ERR_CUDA;
    const LmLayout L = lm_layout(B, K, V, d, sms);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < L.total) return FEF_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int rows = B * K;
    const double c = 1.4426950408889634074 / static_cast<double>(temperature);

    if (device_status && cudaMemsetAsync(device_status, 0, sizeof(int32_t), stream) != cudaSuccess) return FEF_ERR_CUDA;

    // 1. both products with the softmax partials in the epilogue (target rows, then draft rows)
    GemmParams G = {};
    G.tiles_per_chunk = stats_tiles_per_chunk(rows, V, sms);
    G.c = static_cast<float>(c);
    G.tokens = draft_tokens;
    G.row_len = row_len;
    G.K = K;
    G.partials = reinterpret_cast<ChunkPartial*>(ws + L.partials);
    G.logit_at_token = reinterpret_cast<float*>(ws + L.lx);
    G.status = device_status;
    cudaError_t e = launch_gemm<kStats>(target_hidden, draft_hidden, rows, weight, V, d, G, dev, sms, stream);
    if (e != cudaSuccess) return FEF_ERR_CUDA;

    // 2. acceptance tests, first rejection, outputs of the accepted positions, gather of the rejected rows
    AcceptParams A = {};
    A.B = B;
    A.K = K;
    A.V = V;
    A.chunks = L.chunks;
    A.rows = rows;
    A.d = d;
    A.c = static_cast<float>(c);
    A.partials = G.partials;
    A.logit_at_token = G.logit_at_token;
    A.tokens = draft_tokens;
    A.row_len = row_len;
    A.target_hidden = static_cast<const uint16_t*>(target_hidden);
    A.draft_hidden = static_cast<const uint16_t*>(draft_hidden);
    A.gathered = reinterpret_cast<uint16_t*>(ws + L.gathered);
    A.seed = seed;
    A.step = step;
    A.accept_len = accept_len;
    A.out_tokens = tokens;
    A.conf = conf;
    A.tasks = reinterpret_cast<ResidualTask*>(ws + L.tasks);
    A.status = device_status;
    e = launch_pdl(lmhead_accept_kernel, dim3(B), dim3(kAcceptThreads), 0, stream, A);
    if (e != cudaSuccess) return FEF_ERR_CUDA;

    // 3. logits of the rejected positions (2 B rows) in binary32
    GemmParams S = {};
    S.c = 1.f;
    S.K = 1;
    S.logits_out = reinterpret_cast<float*>(ws + L.logits);
    S.ldo = L.ldo;
    S.status = device_status;
    e = launch_gemm<kStore>(ws + L.gathered, nullptr, 2 * B, weight, V, d, S, dev, sms, stream);
    if (e != cudaSuccess) return FEF_ERR_CUDA;

    // 4. residual draw on those rows
    VerifyParams P = {};
    P.geo.B = B;
    P.geo.K = K;
    P.geo.V = V;
    P.geo.vec_elems = V / 4 * 4;
    P.geo.vec_bytes = P.geo.vec_elems * 4;
    P.geo.ld_bytes = L.ldo * 4;
    float c_hi = static_cast<float>(c);
    if (static_cast<double>(c_hi) >= c) c_hi = nextafterf(c_hi, 0.0f);
    P.c_hi = c_hi;
    P.c_lo = static_cast<float>(c - static_cast<double>(c_hi));
    P.c_exact = c;
    if (!(P.c_lo > 0.f) || !(P.c_hi > 0.f)) return FEF_ERR_INVALID_ARG;
    P.wait_limit_ns = kWaitLimitNs;
    P.withhold_stage = -1;
    P.seed = seed;
    P.keys = philox_round_keys(seed);
    P.step = step;
    P.tokens = tokens;
    P.conf = conf;
    P.tasks = A.tasks;
    P.candidates = reinterpret_cast<Candidate*>(ws + L.candidates);
    P.status = device_status;
    const int nvec = P.geo.vec_elems / 4;
    int parts = (2 * sms) / B;
    const int most = (nvec + kResidualThreads * 4 - 1) / (kResidualThreads * 4);
    if (parts > most) parts = most;
    if (parts > kMaxResidualCtas) parts = kMaxResidualCtas;
    if (parts < 1) parts = 1;
    P.geo.residual_ctas = parts;
    e = launch_pdl(lmhead_residual_kernel, dim3(parts, B), dim3(kResidualThreads), 0, stream, P,
                   static_cast<const float*>(S.logits_out), L.ldo);
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

}  // extern "C"

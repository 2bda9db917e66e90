// Bookkeeping of the paper's full-sequence decoding loop (Algorithm 2) on the device, so that a
// decode loop around fef_draft_sample / fef_spec_verify / fef_remask_select needs no host copy
// of its state: the ordered set of unresolved positions and the window b = min{k, L_t}; the
// verification inputs X^(j_m) (verified prefix + draft prefix); the write-back of accepted and
// corrected tokens with their confidences into X and C^(s); the re-masking of LowConf's choice.
// All integer work, a few KB to a few MB per call.
#include <cuda_runtime.h>
#include <stdint.h>

#include "fef.h"

namespace fef {

constexpr int kLoopThreads = 256;

// One CTA per batch row: the first K masked positions in increasing order.
__global__ void __launch_bounds__(kLoopThreads) next_window_kernel(const int32_t* __restrict__ tokens, int L, int K,
                                                                   int32_t* __restrict__ window_pos,
                                                                   int32_t* __restrict__ row_len,
                                                                   int32_t* __restrict__ unresolved) {
    cudaGridDependencySynchronize();  // launched while its predecessor on the stream drains
    __shared__ int s_warp[kLoopThreads / 32];
    const int b = blockIdx.x;
    const int32_t* row = tokens + static_cast<int64_t>(b) * L;
    const int per = (L + kLoopThreads - 1) / kLoopThreads;  // consecutive positions per thread
    const int begin = min(static_cast<int>(threadIdx.x) * per, L), end = min(begin + per, L);
    int mine = 0;
    for (int j = begin; j < end; ++j) mine += row[j] == FEF_MASK_TOKEN;
    // exclusive scan of the threads' counts
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int base = 0, total = 0;
    for (int w = 0; w < kLoopThreads / 32; ++w) {
        if (w < warp) base += s_warp[w];
        total += s_warp[w];
    }
    int rank = base + incl - mine;
    for (int j = begin; j < end && rank < K; ++j)
        if (row[j] == FEF_MASK_TOKEN) window_pos[static_cast<int64_t>(b) * K + rank++] = j;
    const int n = total < K ? total : K;
    for (int t = n + threadIdx.x; t < K; t += kLoopThreads) window_pos[static_cast<int64_t>(b) * K + t] = -1;
    if (threadIdx.x == 0) {
        row_len[b] = n;
        unresolved[b] = total;
    }
}

// One CTA per (b, m): X^(j_m) = the sequence with the drafts of j_0 .. j_{m-1} written in.
__global__ void __launch_bounds__(kLoopThreads) inputs_kernel(const int32_t* __restrict__ tokens,
                                                              const int32_t* __restrict__ window_pos,
                                                              const int32_t* __restrict__ row_len,
                                                              const int32_t* __restrict__ draft_tokens, int L, int K,
                                                              int32_t* __restrict__ inputs) {
    cudaGridDependencySynchronize();  // launched while its predecessor on the stream drains
    const int b = blockIdx.x / K, m = blockIdx.x - b * K;
    const int32_t* row = tokens + static_cast<int64_t>(b) * L;
    int32_t* out = inputs + static_cast<int64_t>(blockIdx.x) * L;
    for (int j = threadIdx.x; j < L; j += kLoopThreads) out[j] = row[j];
    __syncthreads();
    const int upto = min(m, row_len[b]);
    for (int t = threadIdx.x; t < upto; t += kLoopThreads) {
        const int j = window_pos[static_cast<int64_t>(b) * K + t];
        if (j >= 0 && j < L) out[j] = draft_tokens[static_cast<int64_t>(b) * K + t];  // a corrupt position is skipped
    }
}

// One thread per (b, t): write back the committed positions of one verification call.
__global__ void commit_kernel(const int32_t* __restrict__ window_pos, const int32_t* __restrict__ row_len,
                              const int32_t* __restrict__ accept_len, const int32_t* __restrict__ out_tokens,
                              const float* __restrict__ out_conf, int B, int L, int K, int32_t* __restrict__ tokens,
                              float* __restrict__ conf, uint8_t* __restrict__ in_step,
                              int32_t* __restrict__ committed) {
    cudaGridDependencySynchronize();  // launched while its predecessor on the stream drains
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * K) return;
    const int b = idx / K, t = idx - b * K;
    const int a = accept_len[b], n = row_len[b];
    const int m = a < 0 ? -1 : min(a + 1, n);  // accepted drafts plus the corrected position
    if (t == 0) committed[b] = m;
    const int j = window_pos[idx];
    if (t < m && j >= 0 && j < L) {
        const int64_t at = static_cast<int64_t>(b) * L + j;
        tokens[at] = out_tokens[idx];
        conf[at] = out_conf[idx];
        in_step[at] = 1;
    }
}

// Re-corrupt the selected positions (absorbing state: back to MASK) and empty C^(s).
__global__ void remask_apply_kernel(const int32_t* __restrict__ positions, const int32_t* __restrict__ count, int L,
                                    int k, int32_t* __restrict__ tokens, float* __restrict__ conf,
                                    uint8_t* __restrict__ in_step) {
    cudaGridDependencySynchronize();  // launched while its predecessor on the stream drains
    const int b = blockIdx.x;
    for (int j = threadIdx.x; j < L; j += blockDim.x) in_step[static_cast<int64_t>(b) * L + j] = 0;
    const int n = min(count[b], k);
    for (int t = threadIdx.x; t < n; t += blockDim.x) {
        const int j = positions[static_cast<int64_t>(b) * k + t];
        if (j < 0 || j >= L) continue;
        const int64_t at = static_cast<int64_t>(b) * L + j;
        tokens[at] = FEF_MASK_TOKEN;
        conf[at] = -1.0f;
    }
}

// The round counter that fef_draft_sample_at_round / fef_spec_verify_at_round read: plus one,
// unless `unresolved` is given and no row has an unresolved position left (a replayed round
// that had nothing to do takes no number).
__global__ void __launch_bounds__(kLoopThreads) advance_round_kernel(uint32_t* round, const int32_t* unresolved, int B) {
    cudaGridDependencySynchronize();  // launched while its predecessor on the stream drains
    int any = unresolved ? 0 : 1;
    if (unresolved)
        for (int b = threadIdx.x; b < B; b += kLoopThreads) any |= unresolved[b] > 0;
    any = __syncthreads_or(any);
    if (threadIdx.x == 0 && any) *round += 1u;
}

// Programmatic dependent launch: the grid may be scheduled while its predecessor on the stream
// drains; every kernel here waits (cudaGridDependencySynchronize) before it touches memory.
template <typename... Args>
static cudaError_t launch_chained(void (*kernel)(Args...), dim3 grid, dim3 block, void* cuda_stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = static_cast<cudaStream_t>(cuda_stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

static bool loop_sizes_ok(int B, int L, int K) {
    return B >= 1 && B <= FEF_MAX_B && L >= 1 && L <= (1 << 24) && K >= 1 && K <= FEF_MAX_K;
}

}  // namespace fef

extern "C" {

fef_status fef_loop_next_window(const int32_t* tokens, int B, int L, int K, int32_t* window_pos, int32_t* row_len,
                                int32_t* unresolved, void* cuda_stream) {
    using namespace fef;
    if (!tokens || !window_pos || !row_len || !unresolved || !loop_sizes_ok(B, L, K)) return FEF_ERR_INVALID_ARG;
    return fef::launch_chained(fef::next_window_kernel, dim3(B), dim3(kLoopThreads), cuda_stream, tokens, L, K, window_pos, row_len, unresolved) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_loop_verification_inputs(const int32_t* tokens, const int32_t* window_pos, const int32_t* row_len,
                                        const int32_t* draft_tokens, int B, int L, int K, int32_t* inputs,
                                        void* cuda_stream) {
    using namespace fef;
    if (!tokens || !window_pos || !row_len || !draft_tokens || !inputs || !loop_sizes_ok(B, L, K))
        return FEF_ERR_INVALID_ARG;
    return fef::launch_chained(fef::inputs_kernel, dim3(B * K), dim3(kLoopThreads), cuda_stream, tokens, window_pos, row_len, draft_tokens, L, K, inputs) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_loop_commit(const int32_t* window_pos, const int32_t* row_len, const int32_t* accept_len,
                           const int32_t* out_tokens, const float* out_conf, int B, int L, int K, int32_t* tokens,
                           float* conf, uint8_t* in_step, int32_t* committed, void* cuda_stream) {
    using namespace fef;
    if (!window_pos || !row_len || !accept_len || !out_tokens || !out_conf || !tokens || !conf || !in_step ||
        !committed || !loop_sizes_ok(B, L, K))
        return FEF_ERR_INVALID_ARG;
    const int threads = 256, blocks = (B * K + threads - 1) / threads;
    return fef::launch_chained(fef::commit_kernel, dim3(blocks), dim3(threads), cuda_stream, window_pos, row_len, accept_len, out_tokens, out_conf, B, L, K, tokens, conf, in_step, committed) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_loop_remask(const int32_t* positions, const int32_t* count, int B, int L, int k, int32_t* tokens,
                           float* conf, uint8_t* in_step, void* cuda_stream) {
    using namespace fef;
    if (!count || !tokens || !conf || !in_step || k < 0 || (k > 0 && !positions) || !loop_sizes_ok(B, L, 1))
        return FEF_ERR_INVALID_ARG;
    return fef::launch_chained(fef::remask_apply_kernel, dim3(B), dim3(256), cuda_stream, positions, count, L, k, tokens, conf, in_step) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_loop_advance_round(uint32_t* device_round, const int32_t* unresolved, int B, void* cuda_stream) {
    if (!device_round || (unresolved && (B < 1 || B > FEF_MAX_B))) return FEF_ERR_INVALID_ARG;
    return fef::launch_chained(fef::advance_round_kernel, dim3(1), dim3(fef::kLoopThreads), cuda_stream, device_round, unresolved, B) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

}  // extern "C"

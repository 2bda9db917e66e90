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
                                    uint8_t* __restrict__ in_step, const int32_t* __restrict__ gate) {
    cudaGridDependencySynchronize();  // launched while its predecessor on the stream drains
    if (gate && *gate == 0) return;  // (device-driven loop: not the end of a denoising step)
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

// Device-driven loop: what happens after the window of a round is known.  All rows resolved and
// denoising steps left: this round starts with the re-masking (gate = 1, one step fewer).  All rows
// resolved and no step left: the loop's body runs for the last time.  `keep_going` is the condition
// of the graph's WHILE node.
__global__ void __launch_bounds__(kLoopThreads) loop_gate_kernel(const int32_t* __restrict__ unresolved, int B,
                                                                 int32_t* steps_left, int32_t* gate,
                                                                 cudaGraphConditionalHandle keep_going) {
    cudaGridDependencySynchronize();
    int any = 0;
    for (int b = threadIdx.x; b < B; b += kLoopThreads) any |= unresolved[b] > 0;
    any = __syncthreads_or(any);
    if (threadIdx.x == 0) {
        int g = 0;
        unsigned more = 1u;
        if (!any) {
            if (*steps_left > 1) {
                g = 1;
                *steps_left -= 1;
            } else {
                *steps_left = 0;
                more = 0u;
            }
        }
        *gate = g;
        cudaGraphSetConditional(keep_going, more);
    }
}

// Device-driven loop: the round's two status words into the loop's one.
__global__ void merge_status_kernel(const int32_t* __restrict__ a, const int32_t* __restrict__ b, int32_t* out) {
    cudaGridDependencySynchronize();
    if (threadIdx.x == 0 && out) atomicMax(out, max(*a, *b));
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
    return fef::launch_chained(fef::remask_apply_kernel, dim3(B), dim3(256), cuda_stream, positions, count, L, k, tokens, conf, in_step, static_cast<const int32_t*>(nullptr)) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

fef_status fef_loop_advance_round(uint32_t* device_round, const int32_t* unresolved, int B, void* cuda_stream) {
    if (!device_round || (unresolved && (B < 1 || B > FEF_MAX_B))) return FEF_ERR_INVALID_ARG;
    return fef::launch_chained(fef::advance_round_kernel, dim3(1), dim3(fef::kLoopThreads), cuda_stream, device_round, unresolved, B) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}


// ---- the whole loop as one submission
namespace {
struct RunLayout {
    size_t window, row_len, unresolved, draft_tokens, dnorm, tnorm, accept_len, out_tokens, out_conf, committed,
        positions, count, gate, steps_left, status, q, p, draft_ws, verify_ws, total;
    int64_t ld;
};
size_t run_up(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }
bool run_layout(int B, int L, int K, int V, fef_dtype dt, int remask_k, RunLayout* R) {
    if (!fef::loop_sizes_ok(B, L, K) || V < 1 || remask_k < 0 || L > FEF_MAX_REMASK_L) return false;
    if (dt != FEF_F32 && dt != FEF_BF16) return false;
    const int esize = dt == FEF_F32 ? 4 : 2, per_vec = 16 / esize;
    R->ld = (static_cast<int64_t>(V) + per_vec - 1) / per_vec * per_vec;
    const size_t dws = fef_draft_sample_workspace_bytes(B, K, V, dt), vws = fef_spec_verify_workspace_bytes(B, K, V, dt);
    if (dws == 0 || vws == 0) return false;
    const size_t bk = static_cast<size_t>(B) * K;
    size_t at = 0;
    R->window = at; at += run_up(bk * 4);
    R->row_len = at; at += run_up(static_cast<size_t>(B) * 4);
    R->unresolved = at; at += run_up(static_cast<size_t>(B) * 4);
    R->draft_tokens = at; at += run_up(bk * 4);
    R->dnorm = at; at += run_up(bk * 8);
    R->tnorm = at; at += run_up(bk * 8);
    R->accept_len = at; at += run_up(static_cast<size_t>(B) * 4);
    R->out_tokens = at; at += run_up(bk * 4);
    R->out_conf = at; at += run_up(bk * 4);
    R->committed = at; at += run_up(static_cast<size_t>(B) * 4);
    R->positions = at; at += run_up(static_cast<size_t>(B) * (remask_k > 0 ? remask_k : 1) * 4);
    R->count = at; at += run_up(static_cast<size_t>(B) * 4);
    R->gate = at; at += 256;
    R->steps_left = at; at += 256;
    R->status = at; at += 256;
    R->q = at; at += run_up(bk * R->ld * esize);
    R->p = at; at += run_up(bk * R->ld * esize);
    R->draft_ws = at; at += run_up(dws);
    R->verify_ws = at; at += run_up(vws);
    R->total = at;
    return true;
}
}  // namespace

size_t fef_loop_run_synthetic_workspace_bytes(int B, int L, int K, int V, fef_dtype dt, int remask_k) {
    RunLayout R;
    return run_layout(B, L, K, V, dt, remask_k, &R) ? R.total : 0;
}

fef_status fef_loop_run_synthetic(int B, int L, int K, int V, fef_dtype dt, float temperature, uint64_t seed,
                                  int n_steps, int remask_k, float draft_std, float noise_std, float boost_fraction,
                                  float boost, int32_t* tokens, float* conf, uint8_t* in_step, uint32_t* device_round,
                                  void* workspace, size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
    using namespace fef;
    RunLayout R;
    if (!tokens || !conf || !in_step || !device_round || n_steps < 1) return FEF_ERR_INVALID_ARG;
    if (!(temperature > 0.0f)) return FEF_ERR_INVALID_ARG;
    if (!run_layout(B, L, K, V, dt, remask_k, &R)) return FEF_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < R.total) return FEF_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t* steps_left = reinterpret_cast<int32_t*>(ws + R.steps_left);
    int32_t* gate = reinterpret_cast<int32_t*>(ws + R.gate);
    int32_t* round_status = reinterpret_cast<int32_t*>(ws + R.status);
    int32_t* window = reinterpret_cast<int32_t*>(ws + R.window);
    int32_t* row_len = reinterpret_cast<int32_t*>(ws + R.row_len);
    int32_t* unresolved = reinterpret_cast<int32_t*>(ws + R.unresolved);
    int32_t* draft_tokens = reinterpret_cast<int32_t*>(ws + R.draft_tokens);
    double* dnorm = reinterpret_cast<double*>(ws + R.dnorm);
    double* tnorm = reinterpret_cast<double*>(ws + R.tnorm);
    int32_t* accept_len = reinterpret_cast<int32_t*>(ws + R.accept_len);
    int32_t* out_tokens = reinterpret_cast<int32_t*>(ws + R.out_tokens);
    float* out_conf = reinterpret_cast<float*>(ws + R.out_conf);
    int32_t* committed = reinterpret_cast<int32_t*>(ws + R.committed);
    int32_t* positions = reinterpret_cast<int32_t*>(ws + R.positions);
    int32_t* count = reinterpret_cast<int32_t*>(ws + R.count);

    // graph: [steps_left = n_steps, status = 0] -> WHILE(keep_going) { one round }
    cudaGraph_t graph = nullptr, body = nullptr;
    cudaGraphExec_t exec = nullptr;
    cudaStream_t cap = nullptr;
    fef_status result = FEF_ERR_CUDA;
    bool capturing = false;
    do {
        if (cudaGraphCreate(&graph, 0) != cudaSuccess) break;
        cudaGraphConditionalHandle keep_going;
        if (cudaGraphConditionalHandleCreate(&keep_going, graph, 1, cudaGraphCondAssignDefault) != cudaSuccess) break;
        cudaGraphNodeParams cond = {};
        cond.type = cudaGraphNodeTypeConditional;
        cond.conditional.handle = keep_going;
        cond.conditional.type = cudaGraphCondTypeWhile;
        cond.conditional.size = 1;
        cudaGraphNode_t cond_node;
        if (cudaGraphAddNode(&cond_node, graph, nullptr, 0, &cond) != cudaSuccess) break;
        body = cond.conditional.phGraph_out[0];
        if (cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking) != cudaSuccess) break;
        if (cudaStreamBeginCaptureToGraph(cap, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed) != cudaSuccess) break;
        capturing = true;
        fef_status st = fef_loop_next_window(tokens, B, L, K, window, row_len, unresolved, cap);
        if (st == FEF_OK)
            st = launch_chained(loop_gate_kernel, dim3(1), dim3(kLoopThreads), cap, static_cast<const int32_t*>(unresolved), B,
                                steps_left, gate, keep_going) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
        if (st == FEF_OK && remask_k > 0) {
            st = fef_remask_select(conf, in_step, B, L, remask_k, positions, count, cap);
            if (st == FEF_OK)
                st = launch_chained(remask_apply_kernel, dim3(B), dim3(256), cap, static_cast<const int32_t*>(positions),
                                    static_cast<const int32_t*>(count), L, remask_k, tokens, conf, in_step,
                                    static_cast<const int32_t*>(gate)) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
            if (st == FEF_OK) st = fef_loop_next_window(tokens, B, L, K, window, row_len, unresolved, cap);
        }
        if (st == FEF_OK)
            st = fef_synth_logits(ws + R.q, ws + R.p, B, K, V, R.ld, dt, draft_std, noise_std, boost_fraction, boost, seed, 0,
                                  device_round, cap);
        if (st == FEF_OK)
            st = fef_draft_sample_with_target(ws + R.q, ws + R.p, row_len, B, K, V, R.ld, dt, temperature, seed, 0,
                                              device_round, draft_tokens, dnorm, tnorm, ws + R.draft_ws,
                                              R.verify_ws - R.draft_ws, round_status + 1, cap);
        if (st == FEF_OK)
            st = fef_spec_verify_with_norms(ws + R.q, ws + R.p, draft_tokens, dnorm, tnorm, row_len, B, K, V, R.ld, dt,
                                            temperature, seed, 0, device_round, accept_len, out_tokens, out_conf,
                                            ws + R.verify_ws, R.total - R.verify_ws, round_status, cap);
        if (st == FEF_OK)
            st = fef_loop_commit(window, row_len, accept_len, out_tokens, out_conf, B, L, K, tokens, conf, in_step, committed,
                                 cap);
        if (st == FEF_OK) st = fef_loop_advance_round(device_round, unresolved, B, cap);
        if (st == FEF_OK)
            st = launch_chained(merge_status_kernel, dim3(1), dim3(32), cap, static_cast<const int32_t*>(round_status),
                                static_cast<const int32_t*>(round_status + 1), device_status) == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
        cudaGraph_t ended = nullptr;
        const cudaError_t ce = cudaStreamEndCapture(cap, &ended);
        capturing = false;
        if (st != FEF_OK) {
            result = st;
            break;
        }
        if (ce != cudaSuccess) break;
        if (cudaGraphInstantiate(&exec, graph, 0) != cudaSuccess) break;
        const int32_t init_steps = n_steps;
        if (cudaMemcpyAsync(steps_left, &init_steps, sizeof(int32_t), cudaMemcpyHostToDevice, stream) != cudaSuccess) break;
        if (device_status && cudaMemsetAsync(device_status, 0, sizeof(int32_t), stream) != cudaSuccess) break;
        if (cudaGraphLaunch(exec, stream) != cudaSuccess) break;
        if (cudaStreamSynchronize(stream) != cudaSuccess) break;
        result = FEF_OK;
    } while (false);
    if (capturing) {
        cudaGraph_t ended = nullptr;
        cudaStreamEndCapture(cap, &ended);
    }
    if (exec) cudaGraphExecDestroy(exec);
    if (graph) cudaGraphDestroy(graph);
    if (cap) cudaStreamDestroy(cap);
    if (result == FEF_ERR_CUDA) cudaGetLastError();
    return result;
}

}  // extern "C"

// fef_remask_select: LowConf_k of the paper's Algorithm 2 - per batch row, the k
// candidate positions of lowest confidence in (confidence, index) order.
//
// One CTA per batch row.  Every position becomes a 64-bit key
// (order-preserving image of the confidence << 32 | index), non-candidates get
// the largest key.  For k <= 32 (the usual re-mask counts) each warp keeps the
// 32 smallest keys of its share of the row in its lanes (bitonic sort and merge
// by shuffles, no shared memory in the loop) and one warp merges the warps'
// lists; for larger k the keys are sorted in shared memory with a bitonic
// network.  The first min(k, candidates) keys are the answer.
#include <cuda_runtime.h>
#include <stdint.h>

#include "fef.h"

namespace fef {

constexpr int kRemaskThreads = 512;

// Monotone map from binary32 (numeric order, -0 == +0, NaN last) to uint32.
__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t bits = __float_as_uint(f);
    if (f != f) return 0xFFFFFFFEu;
    if (bits == 0x80000000u) bits = 0u;
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}

__global__ void __launch_bounds__(kRemaskThreads) remask_kernel(const float* __restrict__ conf,
                                                               const uint8_t* __restrict__ mask, int L, int k,
                                                               int n_sort, int32_t* __restrict__ positions,
                                                               int32_t* __restrict__ count) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t* keys = reinterpret_cast<uint64_t*>(smem_raw);
    cudaGridDependencySynchronize();  // conf may come straight from a verification call on this stream
    const int b = blockIdx.x;
    const float* c = conf + static_cast<int64_t>(b) * L;
    const uint8_t* m = mask + static_cast<int64_t>(b) * L;

    int mine = 0;
    for (int i = threadIdx.x; i < n_sort; i += kRemaskThreads) {
        uint64_t key = ~0ull;
        if (i < L && m[i] != 0) {
            key = (static_cast<uint64_t>(order_key(c[i])) << 32) | static_cast<uint32_t>(i);
            ++mine;
        }
        keys[i] = key;
    }
    __shared__ int s_total;
    if (threadIdx.x == 0) s_total = 0;
    __syncthreads();
    if (mine) atomicAdd(&s_total, mine);

    for (int size = 2; size <= n_sort; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < (n_sort >> 1); t += kRemaskThreads) {
                const int lo = ((t / stride) * stride << 1) + (t % stride);
                const int hi = lo + stride;
                const bool ascending = ((lo & size) == 0);
                const uint64_t a = keys[lo], z = keys[hi];
                if ((a > z) == ascending) {
                    keys[lo] = z;
                    keys[hi] = a;
                }
            }
        }
    }
    __syncthreads();

    const int total = s_total;
    const int n = total < k ? total : k;
    for (int t = threadIdx.x; t < k; t += kRemaskThreads)
        positions[static_cast<int64_t>(b) * k + t] = t < n ? static_cast<int32_t>(keys[t] & 0xFFFFFFFFu) : -1;
    if (threadIdx.x == 0) count[b] = n;
}

// ---- k <= 32: warp-level selection
constexpr int kSmallThreads = 256;
constexpr int kSmallWarps = kSmallThreads / 32;

// Ascending bitonic sort of the warp's 32 keys (one per lane).
__device__ __forceinline__ uint64_t warp_sort32(uint64_t v, int lane) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const uint64_t other = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
            const bool ascending = (lane & size) == 0;
            const bool lower = (lane & stride) == 0;
            const uint64_t lo = v < other ? v : other, hi = v < other ? other : v;
            v = (lower == ascending) ? lo : hi;
        }
    }
    return v;
}
// The 32 smallest of two ascending lists (a, b: one key per lane each), ascending again.
__device__ __forceinline__ uint64_t warp_merge_low32(uint64_t a, uint64_t b, int lane) {
    const uint64_t reversed = __shfl_sync(0xFFFFFFFFu, b, 31 - lane);
    uint64_t v = a < reversed ? a : reversed;  // bitonic, holds the 32 smallest of the union
#pragma unroll
    for (int stride = 16; stride > 0; stride >>= 1) {
        const uint64_t other = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
        const uint64_t lo = v < other ? v : other, hi = v < other ? other : v;
        v = (lane & stride) == 0 ? lo : hi;
    }
    return v;
}

__global__ void __launch_bounds__(kSmallThreads) remask_small_kernel(const float* __restrict__ conf,
                                                                     const uint8_t* __restrict__ mask, int L, int k,
                                                                     int32_t* __restrict__ positions,
                                                                     int32_t* __restrict__ count) {
    __shared__ uint64_t s_keys[kSmallWarps][32];
    __shared__ int s_total;
    cudaGridDependencySynchronize();  // conf may come straight from a verification call on this stream
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* c = conf + static_cast<int64_t>(b) * L;
    const uint8_t* m = mask + static_cast<int64_t>(b) * L;
    if (threadIdx.x == 0) s_total = 0;
    __syncthreads();

    uint64_t best = ~0ull;  // the warp's 32 smallest keys so far, ascending over the lanes
    int mine = 0;
    for (int base = warp * 32; base < L; base += kSmallThreads) {
        const int i = base + lane;
        uint64_t key = ~0ull;
        if (i < L && m[i] != 0) {
            key = (static_cast<uint64_t>(order_key(c[i])) << 32) | static_cast<uint32_t>(i);
            ++mine;
        }
        best = warp_merge_low32(best, warp_sort32(key, lane), lane);
    }
    mine += __shfl_xor_sync(0xFFFFFFFFu, mine, 16);
    mine += __shfl_xor_sync(0xFFFFFFFFu, mine, 8);
    mine += __shfl_xor_sync(0xFFFFFFFFu, mine, 4);
    mine += __shfl_xor_sync(0xFFFFFFFFu, mine, 2);
    mine += __shfl_xor_sync(0xFFFFFFFFu, mine, 1);
    if (lane == 0 && mine) atomicAdd(&s_total, mine);
    s_keys[warp][lane] = best;
    __syncthreads();
    if (warp != 0) return;
    for (int w = 1; w < kSmallWarps; ++w) best = warp_merge_low32(best, s_keys[w][lane], lane);
    const int total = s_total;
    const int n = total < k ? total : k;
    if (lane < k) positions[static_cast<int64_t>(b) * k + lane] = lane < n ? static_cast<int32_t>(best & 0xFFFFFFFFu) : -1;
    if (lane == 0) count[b] = n;
}

static bool g_remask_attr_done[64];

}  // namespace fef

extern "C" fef_status fef_remask_select(const float* conf, const uint8_t* mask, int B, int L, int k,
                                         int32_t* positions, int32_t* count, void* cuda_stream) {
    using namespace fef;
    if (!conf || !mask || !count || B < 1 || L < 1 || L > FEF_MAX_REMASK_L || k < 0) return FEF_ERR_INVALID_ARG;
    if (k > 0 && !positions) return FEF_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FEF_ERR_CUDA;
    // programmatic dependent launch: the grid may be scheduled while the previous kernel on the
    // stream drains; the kernel waits for it before reading anything
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B);
    cfg.stream = static_cast<cudaStream_t>(cuda_stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (k <= 32) {
        cfg.blockDim = dim3(kSmallThreads);
        cfg.dynamicSmemBytes = 0;
        const cudaError_t e = cudaLaunchKernelEx(&cfg, remask_small_kernel, conf, mask, L, k, positions, count);
        return e == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
    }
    int n_sort = 2;
    while (n_sort < L) n_sort <<= 1;
    const size_t smem = static_cast<size_t>(n_sort) * sizeof(uint64_t);
    if (smem > 48 * 1024 && !g_remask_attr_done[dev]) {
        if (cudaFuncSetAttribute(remask_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 FEF_MAX_REMASK_L * static_cast<int>(sizeof(uint64_t))) != cudaSuccess)
            return FEF_ERR_CUDA;
        g_remask_attr_done[dev] = true;
    }
    cfg.blockDim = dim3(kRemaskThreads);
    cfg.dynamicSmemBytes = smem;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, remask_kernel, conf, mask, L, k, n_sort, positions, count);
    return e == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

static size_t remask_up256(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }

extern "C" size_t fef_remask_select_host_arena_bytes(int B, int L, int k) {
    if (B < 1 || L < 1 || L > FEF_MAX_REMASK_L || k < 0) return 0;
    const size_t n = static_cast<size_t>(B);
    return remask_up256(n * L * 4) + remask_up256(n * L) + remask_up256(n * (k > 0 ? k : 1) * 4) + remask_up256(n * 4);
}

extern "C" fef_status fef_remask_select_host(const float* conf, const uint8_t* mask, int B, int L, int k,
                                              int32_t* positions, int32_t* count, void* device_arena,
                                              size_t device_arena_bytes, void* cuda_stream) {
    if (!conf || !mask || !count || B < 1 || L < 1 || L > FEF_MAX_REMASK_L || k < 0) return FEF_ERR_INVALID_ARG;
    if (k > 0 && !positions) return FEF_ERR_INVALID_ARG;
    const size_t need = fef_remask_select_host_arena_bytes(B, L, k);
    if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255) || device_arena_bytes < need)
        return FEF_ERR_WORKSPACE;
    const size_t n = static_cast<size_t>(B);
    char* d = static_cast<char*>(device_arena);
    float* d_conf = reinterpret_cast<float*>(d);
    uint8_t* d_mask = reinterpret_cast<uint8_t*>(d + remask_up256(n * L * 4));
    int32_t* d_pos = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(d_mask) + remask_up256(n * L));
    int32_t* d_cnt = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(d_pos) + remask_up256(n * (k > 0 ? k : 1) * 4));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(d_conf, conf, n * L * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(d_mask, mask, n * L, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return FEF_ERR_CUDA;
    const fef_status st = fef_remask_select(d_conf, d_mask, B, L, k, d_pos, d_cnt, cuda_stream);
    if (st != FEF_OK) return st;
    if ((k > 0 && cudaMemcpyAsync(positions, d_pos, n * k * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess) ||
        cudaMemcpyAsync(count, d_cnt, n * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
        return FEF_ERR_CUDA;
    return FEF_OK;
}

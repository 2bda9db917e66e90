// fef_synth_logits: seeded synthetic draft and target logits made on the device, for benchmarks and
// tests of the decoding loop (they stand in for the two model calls of Algorithm 2; none of the
// verification's arithmetic is here).  Every element is a pure function of (seed, round, row, id):
//   draft  = draft_std * N(0, 1)  (+ boost with probability boost_512 / 512)
//   target = draft + noise_std * N(0, 1)
// both rounded to the storage type.  Normal deviates: Box-Muller on Philox4x32-10 words, one call
// per two vocabulary ids (counter ((3 << 30) | id / 2, row, round, tag)); the boost bits are the low
// nine bits of the first two words, which the uniforms do not use.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"

namespace fef {

constexpr uint32_t kStreamSynth = 3u;
constexpr int kSynthThreads = 256;

struct SynthParams {
    char* draft;
    char* target;
    int64_t rows, ld_bytes;
    int V;
    float draft_std, noise_std, boost;
    uint32_t boost_512;
    uint64_t seed;
    uint32_t round;
    const uint32_t* device_round;
};

__device__ __forceinline__ void box_muller(uint32_t a, uint32_t b, float* n0, float* n1) {
    const float u0 = uniform_from_word(a), u1 = uniform_from_word(b);
    const float r = sqrtf(-2.0f * __logf(u0));
    float s, c;
    __sincosf(6.283185307179586f * u1, &s, &c);
    *n0 = r * c;
    *n1 = r * s;
}

template <int DT>
__global__ void __launch_bounds__(kSynthThreads) synth_kernel(const __grid_constant__ SynthParams P) {
    cudaGridDependencySynchronize();
    constexpr int N = Elem<DT>::kPerVec;  // ids per 16-byte vector
    const int vec_per_row = (P.V + N - 1) / N;
    const uint32_t round = P.round + (P.device_round ? __ldg(P.device_round) : 0u);
    const uint2 key = make_uint2(static_cast<uint32_t>(P.seed), static_cast<uint32_t>(P.seed >> 32));
    const int64_t total = P.rows * vec_per_row;
    for (int64_t item = static_cast<int64_t>(blockIdx.x) * kSynthThreads + threadIdx.x; item < total;
         item += static_cast<int64_t>(gridDim.x) * kSynthThreads) {
        const int64_t row = item / vec_per_row;
        const int vec = static_cast<int>(item - row * vec_per_row);
        float q[N], p[N];
#pragma unroll
        for (int j = 0; j < N / 2; ++j) {
            const int x = vec * N + 2 * j;
            const uint4 w = philox4x32_10(make_uint4((kStreamSynth << 30) | (static_cast<uint32_t>(x) >> 1),
                                                     static_cast<uint32_t>(row), round, 0x53594E54u), key);
            float d0, d1, e0, e1;
            box_muller(w.x, w.y, &d0, &d1);
            box_muller(w.z, w.w, &e0, &e1);
            q[2 * j] = d0 * P.draft_std + ((w.x & 511u) < P.boost_512 ? P.boost : 0.f);
            q[2 * j + 1] = d1 * P.draft_std + ((w.y & 511u) < P.boost_512 ? P.boost : 0.f);
            p[2 * j] = q[2 * j] + e0 * P.noise_std;
            p[2 * j + 1] = q[2 * j + 1] + e1 * P.noise_std;
        }
        char* qrow = P.draft + row * P.ld_bytes;
        char* prow = P.target + row * P.ld_bytes;
        if constexpr (DT == FEF_F32) {
            // (the row pitch covers whole vectors: entries between V and the pitch are written too)
            *reinterpret_cast<float4*>(qrow + static_cast<int64_t>(vec) * 16) = make_float4(q[0], q[1], q[2], q[3]);
            *reinterpret_cast<float4*>(prow + static_cast<int64_t>(vec) * 16) = make_float4(p[0], p[1], p[2], p[3]);
        } else {
            uint32_t qw[4], pw[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // round to nearest even into the upper halves
                const __nv_bfloat162 qb = __floats2bfloat162_rn(q[2 * j], q[2 * j + 1]);
                const __nv_bfloat162 pb = __floats2bfloat162_rn(p[2 * j], p[2 * j + 1]);
                qw[j] = *reinterpret_cast<const uint32_t*>(&qb);
                pw[j] = *reinterpret_cast<const uint32_t*>(&pb);
            }
            *reinterpret_cast<uint4*>(qrow + static_cast<int64_t>(vec) * 16) = make_uint4(qw[0], qw[1], qw[2], qw[3]);
            *reinterpret_cast<uint4*>(prow + static_cast<int64_t>(vec) * 16) = make_uint4(pw[0], pw[1], pw[2], pw[3]);
        }
    }
}

}  // namespace fef

extern "C" fef_status fef_synth_logits(void* draft_logits, void* target_logits, int B, int K, int V, int64_t ld,
                                       fef_dtype dt, float draft_std, float noise_std, float boost_fraction,
                                       float boost, uint64_t seed, uint32_t round, const uint32_t* device_round,
                                       void* cuda_stream) {
    using namespace fef;
    if (dt != FEF_F32 && dt != FEF_BF16) return FEF_ERR_DTYPE;
    if (!draft_logits || !target_logits || B < 1 || K < 1 || V < 1 || ld < V) return FEF_ERR_INVALID_ARG;
    if (!(boost_fraction >= 0.f) || boost_fraction > 1.f) return FEF_ERR_INVALID_ARG;
    const int esize = dt == FEF_F32 ? 4 : 2, per_vec = 16 / esize;
    if ((reinterpret_cast<uintptr_t>(draft_logits) & 15) || (reinterpret_cast<uintptr_t>(target_logits) & 15) ||
        ((ld * esize) & 15))
        return FEF_ERR_ALIGNMENT;
    if (ld < (static_cast<int64_t>(V) + per_vec - 1) / per_vec * per_vec) return FEF_ERR_INVALID_ARG;  // whole vectors are written
    int dev = -1, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return FEF_ERR_CUDA;
    SynthParams P;
    P.draft = static_cast<char*>(draft_logits);
    P.target = static_cast<char*>(target_logits);
    P.rows = static_cast<int64_t>(B) * K;
    P.ld_bytes = ld * esize;
    P.V = V;
    P.draft_std = draft_std;
    P.noise_std = noise_std;
    P.boost = boost;
    P.boost_512 = static_cast<uint32_t>(boost_fraction * 512.0f + 0.5f);
    P.seed = seed;
    P.round = round;
    P.device_round = device_round;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sms * 8));
    cfg.blockDim = dim3(kSynthThreads);
    cfg.stream = static_cast<cudaStream_t>(cuda_stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = dt == FEF_F32 ? cudaLaunchKernelEx(&cfg, synth_kernel<FEF_F32>, P)
                                        : cudaLaunchKernelEx(&cfg, synth_kernel<FEF_BF16>, P);
    return e == cudaSuccess ? FEF_OK : FEF_ERR_CUDA;
}

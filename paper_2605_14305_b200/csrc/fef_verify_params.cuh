// Parameter block of a verification call, shared by the kernels of fef_verify.cu and by the
// residual draw (fef_residual.cuh), which the hidden-state entry point reuses.
#pragma once

#include <stdint.h>

#include "fef.h"
#include "fef_common.cuh"

namespace fef {

// Work split of one call, computed on the host and passed by value to the kernels.
struct Geometry {
    int B, K, V;
    int units_per_row;    // 2: target row and draft row; 1 when only the target rows are streamed (greedy
                          // mode, or the draft laws' normalisers are given)
    int tile_bytes;       // bytes of one streaming tile (8, 16, 32 or 64 KiB)
    int vec_bytes;        // bytes of a row covered by whole 16-byte vectors
    int vec_elems;        // the same in elements; elements beyond are the row's "tail"
    int tiles_per_unit;   // tiles per row (0 when a row holds no whole vector)
    int tiles_per_claim;  // tiles one claim covers
    int claims_per_unit;  // claims per row (>= 1, also for rows without a whole vector)
    int grid;             // CTAs of the streaming kernel
    int warp_per_row;     // 1: short rows, many of them: rows_kernel (one warp per row) streams instead
    int residual_ctas;    // CTAs per rejected row in the residual kernel
    int small;            // 1: few rows: small_rows_kernel with (small_parts, B) CTAs streams instead of stream_kernel
    int small_parts;
    int small_group;      // ... in which this many consecutive warps share a row: 1, 2, 4 or 8 (a whole CTA)
    int small_ctas_per_row;  // ... and, with whole CTAs, this many CTAs (one thread-block cluster) share a row; else 1
    int64_t num_units;    // rows to stream: B * K * units_per_row
    int64_t num_claims;   // num_units * claims_per_unit
    int64_t ld_bytes;     // row pitch in bytes
};

struct VerifyParams {
    Geometry geo;
    const char* target;   // p logits
    const char* draft;    // q logits
    const int32_t* draft_tokens;
    const int32_t* row_len;
    const double* draft_norm;  // [B*K] log2 normalisers of the draft laws, or null: stream the draft rows
    const double* target_norm; // [B*K] log2 normalisers of the target laws, or null (given only together with draft_norm:
                               // then nothing is streamed)
    float c_hi, c_lo;     // log2(e)/T split in two binary32 numbers, c_lo > 0 (or 0 for bfloat16)
    double c_exact;       // log2(e)/T in double precision (the double-precision pass of the residual draw)
    unsigned long long wait_limit_ns;  // how long a wait inside the streaming kernel may last
    int withhold_stage;   // test builds only: CTA 0 never delivers its stage of this number (-1: none)
    uint64_t seed;
    uint32_t step;
    const uint32_t* round; // device word added to `step` when the kernels run, or null
    PhiloxKeys keys;       // round keys of `seed`
    int32_t* accept_len;
    int32_t* tokens;
    float* conf;
    Control* ctl;          // cleared by begin_call_kernel
    Partial* partials;     // [num_claims]: unit u owns entries [u * claims_per_unit, ...)
    ResidualTask* tasks;   // [B]
    Candidate* candidates; // [B][residual_ctas][kCandidatesPerCta]
    int vocab_offset;      // global id of element 0 of every row (a multiple of 8; 0 unless the vocabulary is sharded)
    VpCandidate* vp_out;   // [B] vocabulary-parallel mode: the residual kernel reports here instead of committing
    int32_t* status;
};

// The call's step number: the by-value part plus, if given, a device-resident round counter
// (read when the kernel runs, so that a replayed CUDA graph draws fresh random numbers).
__device__ __forceinline__ uint32_t step_of(const VerifyParams& P) {
    return P.step + (P.round ? __ldg(P.round) : 0u);
}

}  // namespace fef

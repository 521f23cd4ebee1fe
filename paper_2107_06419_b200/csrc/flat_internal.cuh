// Internal declarations shared by the translation units of libflat_attn (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/flat_attn.h"

namespace flat {

// A validated attention problem (device pointers).
struct Problem {
    const void* Q; const void* K; const void* V; void* O;
    int B, H, Nq, Nk, d;
    float scale;
    int dtype;
    const int32_t* k_valid_len;
    int32_t* status;
};

// Each launcher enqueues its kernels on `st` and returns a FLAT_* code; *launches (if
// non-null) receives the number of kernels enqueued.
int launch_fused_simt(const Problem& p, cudaStream_t st);
int launch_naive(const Problem& p, void* L, void* A, cudaStream_t st);
int launch_fused_tc(const Problem& p, cudaStream_t st);
int launch_fused_tc2(const Problem& p, cudaStream_t st);

}  // namespace flat

// Internal declarations shared by the translation units of libflat_attn (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

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
    int causal;                      // 0 / 1: query i sees keys j <= i + (Nk - Nq)
    float* lse;                      // optional [B,H,Nq] fp32 output of the fused kernels: log-sum-exp of each row's scaled logits
    // optional additive term of the scaled logits: element (b,h,i,j) at b * bias_sb + h * bias_sh + i * Nk + j
    const void* bias;
    int bias_dtype;                  // FLAT_DTYPE_*
    long long bias_sb, bias_sh;      // strides in elements; 0 = the same values for every batch / head
    // optional pruning map over 128 x 128 blocks of the logit matrix: byte (b,h,tq,tk) at
    // b * bmask_sb + h * bmask_sh + tq * ceil(Nk / 128) + tk; 0 = the block takes no part
    const uint8_t* block_mask;
    long long bmask_sb, bmask_sh;
};

// What a kernel needs to read the bias (passed by value).
struct BiasArg {
    const void* p;
    int f32;                         // 1: float32, 0: bf16
    long long sb, sh;
    int vec;                         // 16-byte loads allowed (base, strides and Nk all multiples of 16 bytes)
};
inline BiasArg bias_arg(const Problem& q) {
    const long long es = q.bias_dtype == FLAT_DTYPE_F32 ? 4 : 2, per16 = 16 / es;
    const bool vec = q.bias && (reinterpret_cast<uintptr_t>(q.bias) & 15u) == 0 && q.Nk % per16 == 0 &&
                     q.bias_sb % per16 == 0 && q.bias_sh % per16 == 0;
    return BiasArg{q.bias, q.bias_dtype == FLAT_DTYPE_F32 ? 1 : 0, q.bias_sb, q.bias_sh, vec ? 1 : 0};
}

// A validated backward problem (device pointers; bf16 tensors, fp32 lse / delta).
struct BwdProblem {
    const void *Q, *K, *V, *O, *dO;
    const float* lse;
    void *dQ, *dK, *dV;
    float* delta;
    int B, H, Nq, Nk, d;
    float scale;
    const int32_t* k_valid_len;
    int32_t* status;
    int causal;
};
int launch_bwd_tc(const BwdProblem& p, cudaStream_t st);   // bf16, d in {64, 128}: two kernels (dQ; dK and dV)

// Argument check of the public parameter block (what every fused / baseline entry point applies
// before it launches anything): FLAT_OK or the error code.
int check_params(const flat_attn_params_t* p);

// Each launcher enqueues its kernels on `st` and returns a FLAT_* code; *launches (if
// non-null) receives the number of kernels enqueued.
int launch_fused_simt(const Problem& p, cudaStream_t st);
int launch_naive(const Problem& p, void* L, void* A, cudaStream_t st);
int launch_fused_tc(const Problem& p, cudaStream_t st);
int launch_fused_tc2(const Problem& p, cudaStream_t st);      // (also the tensor-core kernel for calls with a bias)
// (only_if_resident: sixteen-CTA clusters only when all clusters of the launch can run at the same time; else
// FLAT_ERR_UNSUPPORTED)
int launch_fused_tc2_single(const Problem& p, cudaStream_t st, int key_split = 1, bool only_if_resident = false);
// The same tile worked on by two warpgroups that take alternate key tiles (bf16, d = 64, dense; key_split 1, 2, 4, 8).
int launch_fused_tc2_halves(const Problem& p, cudaStream_t st, int key_split = 1, bool only_if_resident = false);   // (key_split 1, 2, 4, 8, 16)   // (d = 64; with a block mask also d = 128; key_split 2 / 4: the keys of a tile over a CTA cluster)
int launch_fused_tc3(const Problem& p, cudaStream_t st);
// How the last launch_fused_tc3 of this host thread dealt its items (FLAT_SCHEDULE_*; 0 before any).
extern thread_local int g_last_schedule;
bool tf32_applies(const Problem& p);               // fp32, d = 64, no bias, no pruning map
int launch_fused_tf32(const Problem& p, cudaStream_t st);     // fp32 tensors through split tf32 products
bool rgran_applies(const Problem& p);              // bf16, d = 64, Nk <= 512
int launch_fused_rgran(const Problem& p, cudaStream_t st);
// Packed variable-length batches (bf16; fused_tc3: d = 64, fused_tc2: d = 128): Q, O [total_q, H, d], K, V [total_k, H, d].
int launch_fused_tc2_varlen(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_q,
                            const int32_t* cu_k, int num_seqs, int H, int64_t total_q, int64_t total_k,
                            int max_seqlen_q, float scale, int causal, int32_t* status, cudaStream_t st);
int launch_fused_tc3_varlen(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_q,
                            const int32_t* cu_k, int num_seqs, int H, int64_t total_q, int64_t total_k,
                            int max_seqlen_q, float scale, int causal, int32_t* status, cudaStream_t st);
// The activation-weight operators around the fused path (proj_gemm.cu): Q/K/V projection into
// head-major tensors and Output projection out of one.
int launch_qkv_proj(const void* X, const void* Wqkv, void* Q, void* K, void* V, int B, int N, int H, int d, int Dm,
                    int32_t* status, cudaStream_t st);
int launch_out_proj(const void* O, const void* Wo, void* Y, int B, int N, int H, int d, int Dm, int32_t* status,
                    cudaStream_t st);
int launch_fc(const void* X, const void* W, void* Y, int M, int Kdim, int Nout, int32_t* status, cudaStream_t st);
// The block's normalisation layer (layernorm.cu): Y = gamma * normalise(X + R) + beta over rows of D features.
int launch_layernorm(const void* X, const void* R, const void* gamma, const void* beta, void* Y, long long M, int D,
                     float eps, cudaStream_t st);
int launch_wait_timeout_selftest(int32_t* status, cudaStream_t st);
int launch_exp2_poly_selftest(const float* x, float* y, int n, cudaStream_t st);
// Tensor-core versions of the baseline's two contractions (bf16, d in {64,128}, Nk % 8 == 0).
bool naive_tc_applies(const Problem& p);
int launch_naive_logit_tc(const Problem& p, float* L, cudaStream_t st);
int launch_naive_attend_tc(const Problem& p, const void* A, cudaStream_t st);

// Raises the dynamic shared-memory limit of `Kernel` once per device (the attribute is sticky,
// and setting it on every call costs microseconds that small problems notice).
template <auto Kernel>
inline bool ensure_dynamic_smem(size_t bytes) {
    static std::atomic<uint64_t> done{0};               // bit i: set for device ordinal i (< 64)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const uint64_t bit = dev >= 0 && dev < 64 ? (1ull << dev) : 0;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return true;
    if (cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) !=
        cudaSuccess)
        return false;
    if (bit) done.fetch_or(bit, std::memory_order_release);
    return true;
}

// Number of SMs of the current device (cached per host thread); 148 if the query fails.
inline int device_sm_count() {
    thread_local int cached_dev = -1, cached_sms = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return 148;
        cached_dev = dev;
        cached_sms = sms;
    }
    return cached_sms;
}

}  // namespace flat

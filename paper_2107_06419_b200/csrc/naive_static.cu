// flat_attn_naive_fwd_static: the unfused baseline for callers that cannot allocate device
// memory.  The logit and weight tensors live in one file-scope device array that is part of
// the library image, so the call path contains no cudaMalloc/cudaFree and no allocating
// library routine.  (The array becomes resident when the runtime loads this part of the
// library on a device -- at the latest during the first call's address lookup -- which is the
// one moment at which a device short of memory can make the call fail.)
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "flat_internal.cuh"

namespace {

constexpr int64_t kMaxElems = FLAT_STATIC_MAX_ELEMS;                 // B*H*Nq*Nk
constexpr size_t kLBytes = static_cast<size_t>(kMaxElems) * 4;       // fp32 logits
constexpr size_t kABytes = static_cast<size_t>(kMaxElems) * 2;       // bf16 weights
constexpr int kMaxDevices = 64;

// Resident on every GPU that loads the library, until the process exits.  In host code this
// name is only a handle for the runtime's symbol table, not a device address.
static __device__ __align__(256) unsigned char g_scratch[kLBytes + kABytes];

std::mutex g_mu;
void* g_scratch_addr[kMaxDevices];      // device address of g_scratch, per device ordinal
bool g_scratch_ready[kMaxDevices];

// Looks up (once per device, with that device current) where g_scratch lives on the GPU.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FLAT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ready[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr) return FLAT_ERR_CUDA;
        g_scratch_addr[dev] = p;
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_addr[dev];
    return FLAT_OK;
}

}  // namespace

extern "C" int flat_attn_naive_fwd_static(const void* Q, const void* K, const void* V, void* O, int B, int H,
                                          int Nq, int Nk, int d, float scale, void* stream) {
    if (B < 1 || H < 1 || Nq < 1 || Nk < 1) return FLAT_ERR_SHAPE;
    // Size gate first: nothing below runs, and the device is not touched, for a problem that
    // does not fit the built-in scratch.
    int64_t elems = static_cast<int64_t>(B) * H;
    if (elems > kMaxElems) return FLAT_ERR_WORKSPACE;
    elems *= Nq;
    if (elems > kMaxElems) return FLAT_ERR_WORKSPACE;
    elems *= Nk;
    if (elems > kMaxElems) return FLAT_ERR_WORKSPACE;
    // Then the remaining argument rules (pointers, d, alignment, scale), with stand-ins for L and A,
    // so that a bad argument is reported as such before the device is looked at.
    {
        flat_attn_params_t chk{Q, K, V, O, B, H, Nq, Nk, d, scale, FLAT_DTYPE_BF16, nullptr, nullptr, FLAT_VARIANT_AUTO, 0, nullptr, nullptr, 0, 0, 0, nullptr, 0, 0};
        const int rc = flat::check_params(&chk);
        if (rc != FLAT_OK) return rc;
    }
    void* base = nullptr;
    const int rc = scratch_for_current_device(&base);
    if (rc != FLAT_OK) return rc;
    void* L = base;
    void* A = static_cast<unsigned char*>(base) + kLBytes;
    // Same three kernels as flat_attn_naive_fwd; they overwrite every element of L and A that
    // this problem uses, so the previous call's contents never need clearing.
    return flat_attn_naive_fwd(Q, K, V, O, L, A, B, H, Nq, Nk, d, scale, stream);
}

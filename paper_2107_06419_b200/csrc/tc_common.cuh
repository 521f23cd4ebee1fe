// Helpers shared by the tensor-core kernels: bounded mbarrier waits, exp2, bf16 packing, and the
// host-side construction of TMA tensor maps.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

namespace flat {
namespace tc {

constexpr long long WAIT_CYCLES = 2000000000ll;   // ~1 s at 2 GHz
constexpr float RESCALE_THRESHOLD = 8.0f;         // log2 units: P stays <= 2^8

// Waits for the phase of `bar` with the given parity.  Gives up when another role of the CTA has
// raised the abort flag or after WAIT_CYCLES; the first thread to time out raises the flag and
// records `code` in *status.  Never traps, never spins without limit.
__device__ __forceinline__ bool bounded_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                             int32_t* status, int code, long long limit = WAIT_CYCLES) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        // The inner probes cost two instructions each; the clock and the abort flag are looked at
        // once per batch so that a waiting warp leaves the issue slots to the working ones.
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            if (status) atomicExch(status, code);
            return false;
        }
    }
}

// The same wait with the barrier and the abort flag given as 32-bit shared-window addresses.
// SLEEP_NS > 0: the thread sleeps that long between probes -- for a role whose reaction time does
// not matter (a producer that runs ahead of its ring) and that should leave the issue slots and
// the shared-memory pipe to the working warps while it waits.
template <unsigned SLEEP_NS = 0>
__device__ __forceinline__ bool bounded_wait_s(uint32_t bar_addr, uint32_t parity, uint32_t abort_addr,
                                               int32_t* status, int code, long long limit = WAIT_CYCLES) {
    if (ptx::mbar_try_wait_s(bar_addr, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i) {
            if (SLEEP_NS) __nanosleep(SLEEP_NS);
            if (ptx::mbar_try_wait_s(bar_addr, parity)) return true;
        }
        int aborted;
        asm volatile("ld.volatile.shared::cta.s32 %0, [%1];" : "=r"(aborted) : "r"(abort_addr) : "memory");
        if (aborted) return false;
        if (clock64() - t0 > limit) {
            asm volatile("st.volatile.shared::cta.s32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
            if (status) atomicExch(status, code);
            return false;
        }
    }
}

// Teardown helper: wait for a copy this thread started, with a time limit and no side effects.
__device__ __forceinline__ void drain_wait(uint64_t* bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, parity))
        if (clock64() - t0 > WAIT_CYCLES) return;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 2^x on the FMA and integer pipes instead of the ex2 unit: x = r + f with r = round(x) and
// f in [-0.5, 0.5]; 2^f by a cubic (max relative error 7.7e-5, far below the bf16 rounding that
// the weights undergo next) and 2^r by adding r to the exponent field.  x is clamped to
// [-126, 126] so that the exponent arithmetic cannot wrap (the cubic lies in [0.70, 1.42], biased
// exponent 126 or 127, so r >= -126 keeps the field at 0 or above): below, the result is a
// denormal of about 2^-126 (as good as 0 next to a row maximum of order 1); above, it is 2^126,
// which trips the caller's overflow check exactly like the ex2 unit's +inf would.
__device__ __forceinline__ float ex2_poly(float x) {
    x = fminf(fmaxf(x, -126.f), 126.f);
    const float t = x + 12582912.f;                    // 1.5 * 2^23: the low mantissa bits now hold round(x)
    const float r = t - 12582912.f;
    const float f = x - r;
    float p = fmaf(0.05508868f, f, 0.24260405f);
    p = fmaf(p, f, 0.69327624f);
    p = fmaf(p, f, 0.99992894f);
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}

// Three-input maximum / minimum (one instruction on sm_100).
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry-point lookup (no link against libcuda).
inline EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 tensor [BH, N, d] (d contiguous) viewed as 3-D {d, N, BH}; box = 64 x rows x 1, 128-byte swizzle.
inline bool make_map(CUtensorMap* m, const void* ptr, int BH, int N, int d, int box_rows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(BH)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 2, static_cast<cuuint64_t>(N) * d * 2};
    cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A packed tensor [tokens, H, d] bf16 (variable-length batches) as a TMA tensor {d, H, tokens} with
// boxes of 64 features x one head x box_rows tokens (in shared memory: box_rows rows of 128 bytes, as
// for the batched layout).
inline bool make_map_packed(CUtensorMap* m, const void* ptr, int64_t tokens, int H, int d, int box_rows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(tokens)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 2, static_cast<cuuint64_t>(H) * d * 2};
    cuuint32_t box[3] = {64, 1, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace flat

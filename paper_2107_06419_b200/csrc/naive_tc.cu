// The two contractions of the paper's unfused baseline (Section 4.2, Fig. 7(a)) on the tensor
// cores, so that the baseline is limited by what the paper says limits it -- the traffic of the
// [B,H,Nq,Nk] intermediates through device memory -- and not by FFMA throughput:
//   naive_logit_tc_kernel :  L = scale * Q K^T   (bf16 in, fp32 out, one 128x128 tile per CTA)
//   naive_attend_tc_kernel:  O = A V             (A bf16 read through TMA in 128x64 tiles)
// The row softmax between them is naive_softmax_kernel (simt_kernels.cu).
// Conditions: bf16, d in {64, 128}, Nk a multiple of 8 (TMA row pitch of A); otherwise the FFMA
// kernels run.  Every wait is bounded (tc_common.cuh).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flat_internal.cuh"
#include "ptx_sm100.cuh"
#include "tc_common.cuh"

namespace flat {

using namespace ptx;
using namespace tc;

namespace {

constexpr int TM = 128;      // rows per CTA
constexpr int NTHREADS = 192;   // warps 0-3 epilogue, warp 4 TMA, warp 5 MMA issue

// ---------------------------------------------------------------------------------- L = scale Q K^T
template <int D>
__global__ void __launch_bounds__(NTHREADS)
naive_logit_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      float* __restrict__ L, int Nq, int Nk, float scale, int32_t* status) {
    constexpr int TILE_BYTES = TM * D * 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Qs = base;
    uint8_t* Ks = base + TILE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + 2 * TILE_BYTES);     // [0] operands landed, [1] S done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.z, row0 = blockIdx.y * TM, k0 = blockIdx.x * 128;

    if (threadIdx.x == 4 * 32) { mbar_init(&bars[0], 1); mbar_init(&bars[1], 1); *abort_flag = 0; fence_mbar_init(); }
    if (warp == 0) { tmem_alloc(tmem_slot, 128); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        if (elect_one()) {
            mbar_arrive_expect_tx(&bars[0], 2 * TILE_BYTES);
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                tma_load_3d(Qs + c * TM * 128, &tmQ, &bars[0], c * 64, row0, bh);
                tma_load_3d(Ks + c * 128 * 128, &tmK, &bars[0], c * 64, k0, bh);
            }
        }
    } else if (warp == 5) {
        bool ok = __all_sync(0xffffffffu, bounded_wait(&bars[0], 0, abort_flag, status, 0x400));
        if (ok) {
            tc_fence_after();
            if (elect_one()) {
                constexpr uint32_t IDESC = make_idesc_bf16(TM, 128, 0, 0);
                const uint64_t qd = make_smem_desc_sw128(smem_u32(Qs), 16, 1024);
                const uint64_t kd = make_smem_desc_sw128(smem_u32(Ks), 16, 1024);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint64_t off = static_cast<uint64_t>(((k / 4) * (TM * 128) + (k % 4) * 32) >> 4);
                    mma_ss(tmem, qd + off, kd + off, IDESC, k > 0);
                }
                tc_commit(&bars[1]);
            }
            __syncwarp();
        }
    } else {
        bool ok = __all_sync(0xffffffffu, bounded_wait(&bars[1], 0, abort_flag, status, 0x410));
        if (ok) {
            tc_fence_after();
            const int row = row0 + warp * 32 + lane;
            const uint32_t tl = tmem + (static_cast<uint32_t>(warp * 32) << 16);
            float* out = L + (static_cast<int64_t>(bh) * Nq + row) * Nk + k0;
            const bool vec = (Nk & 3) == 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tl + c * 32, r);
                tc_wait_ld();
                if (row < Nq) {
                    if (vec && k0 + c * 32 + 32 <= Nk) {
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            float4 w = make_float4(__uint_as_float(r[4 * v]) * scale, __uint_as_float(r[4 * v + 1]) * scale,
                                                   __uint_as_float(r[4 * v + 2]) * scale, __uint_as_float(r[4 * v + 3]) * scale);
                            *reinterpret_cast<float4*>(out + c * 32 + 4 * v) = w;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (k0 + c * 32 + i < Nk) out[c * 32 + i] = __uint_as_float(r[i]) * scale;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 128);
}

// ---------------------------------------------------------------------------------- O = A V
template <int D> struct AttendLayout {
    static constexpr int STAGES = 4;
    static constexpr int A_BYTES = TM * 64 * 2;          // 128 rows x 64 keys
    static constexpr int V_BYTES = 64 * D * 2;           // 64 keys x d
    static constexpr int TILE_BYTES = STAGES * (A_BYTES + V_BYTES);
    static constexpr int SMEM_BYTES = TILE_BYTES + 256 + 1024;
    static constexpr uint32_t TMEM_COLS = D;             // 64 or 128
};

template <int D>
__global__ void __launch_bounds__(NTHREADS)
naive_attend_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmV,
                       __nv_bfloat16* __restrict__ O, int H, int Nq, int Nk, const int32_t* __restrict__ valid_len,
                       int32_t* status) {
    using LY = AttendLayout<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* As = base;
    uint8_t* Vs = base + LY::STAGES * LY::A_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + LY::TILE_BYTES);     // full[S], empty[S], done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * LY::STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, row0 = blockIdx.x * TM;
    int n = Nk;
    if (valid_len) { n = valid_len[bh / H]; n = n < 0 ? 0 : (n > Nk ? Nk : n); }
    const int ntiles = (n + 63) / 64;                    // weights beyond n are zero: nothing to add

    if (threadIdx.x == 4 * 32) {
        for (int i = 0; i < 2 * LY::STAGES + 1; ++i) mbar_init(&bars[i], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, LY::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    uint64_t* full = bars;
    uint64_t* empty = bars + LY::STAGES;
    uint64_t* done = bars + 2 * LY::STAGES;

    if (warp == 4) {
        if (lane == 0) {
            bool ok = true;
            int issued = 0;
            for (int j = 0; j < ntiles && ok; ++j) {
                const int s = j % LY::STAGES;
                ok = bounded_wait(&empty[s], ((j / LY::STAGES) & 1) ^ 1, abort_flag, status, 0x420);
                if (!ok) break;
                mbar_arrive_expect_tx(&full[s], LY::A_BYTES + LY::V_BYTES);
                tma_load_3d(As + s * LY::A_BYTES, &tmA, &full[s], j * 64, row0, bh);
#pragma unroll
                for (int c = 0; c < D / 64; ++c)
                    tma_load_3d(Vs + s * LY::V_BYTES + c * 64 * 128, &tmV, &full[s], c * 64, j * 64, bh);
                issued = j + 1;
            }
            if (!ok)
                for (int j = issued > LY::STAGES ? issued - LY::STAGES : 0; j < issued; ++j)
                    drain_wait(&full[j % LY::STAGES], (j / LY::STAGES) & 1);
        }
    } else if (warp == 5) {
        constexpr uint32_t IDESC = make_idesc_bf16(TM, D, 0, 1);
        const uint64_t ad = make_smem_desc_sw128(smem_u32(As), 16, 1024);
        const uint64_t vd = make_smem_desc_sw128(smem_u32(Vs), 64 * 128, 1024);
        bool ok = true;
        for (int j = 0; j < ntiles && ok; ++j) {
            const int s = j % LY::STAGES;
            ok = __all_sync(0xffffffffu, bounded_wait(&full[s], (j / LY::STAGES) & 1, abort_flag, status, 0x430));
            if (!ok) break;
            tc_fence_after();
            if (elect_one()) {
                const uint64_t a = ad + static_cast<uint64_t>((s * LY::A_BYTES) >> 4);
                const uint64_t v = vd + static_cast<uint64_t>((s * LY::V_BYTES) >> 4);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    mma_ss(tmem, a + static_cast<uint64_t>((k * 32) >> 4), v + static_cast<uint64_t>((k * 2048) >> 4),
                           IDESC, (j > 0 || k > 0));
                tc_commit(&empty[s]);
                if (j == ntiles - 1) tc_commit(done);
            }
            __syncwarp();
        }
    } else {
        bool ok = true;
        if (ntiles > 0) ok = __all_sync(0xffffffffu, bounded_wait(done, 0, abort_flag, status, 0x440));
        if (ok) {
            tc_fence_after();
            const int row = row0 + warp * 32 + lane;
            const uint32_t tl = tmem + (static_cast<uint32_t>(warp * 32) << 16);
            __nv_bfloat16* orow = O + (static_cast<int64_t>(bh) * Nq + row) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                if (ntiles > 0) {
                    tmem_ld_x32(tl + c * 32, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
                if (row < Nq) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
                        w.y = pack_bf16x2(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                        w.z = pack_bf16x2(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                        w.w = pack_bf16x2(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                        *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = w;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, LY::TMEM_COLS);
}

template <int D>
int launch_logit(const Problem& p, float* L, cudaStream_t st) {
    CUtensorMap tmQ, tmK;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, D, TM) || !make_map(&tmK, p.K, BH, p.Nk, D, 128)) return FLAT_ERR_CUDA;
    constexpr int SMEM = 2 * TM * D * 2 + 256 + 1024;
    if (!ensure_dynamic_smem<naive_logit_tc_kernel<D>>(SMEM)) return FLAT_ERR_CUDA;
    dim3 grid((p.Nk + 127) / 128, (p.Nq + TM - 1) / TM, BH);
    naive_logit_tc_kernel<D><<<grid, NTHREADS, SMEM, st>>>(tmQ, tmK, L, p.Nq, p.Nk, p.scale, p.status);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

template <int D>
int launch_attend(const Problem& p, const void* A, cudaStream_t st) {
    using LY = AttendLayout<D>;
    CUtensorMap tmA, tmV;
    const int BH = p.B * p.H;
    // A viewed as [BH, Nq, Nk] bf16 (Nk contiguous): boxes of 64 keys x 128 rows; V boxes of 64 x 64.
    if (!make_map(&tmA, A, BH, p.Nq, p.Nk, TM) || !make_map(&tmV, p.V, BH, p.Nk, D, 64)) return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<naive_attend_tc_kernel<D>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
    dim3 grid((p.Nq + TM - 1) / TM, BH);
    naive_attend_tc_kernel<D><<<grid, NTHREADS, LY::SMEM_BYTES, st>>>(
        tmA, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, p.k_valid_len, p.status);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

}  // namespace

bool naive_tc_applies(const Problem& p) {
    return p.dtype == FLAT_DTYPE_BF16 && (p.d == 64 || p.d == 128) && (p.Nk % 8) == 0;
}

int launch_naive_logit_tc(const Problem& p, float* L, cudaStream_t st) {
    return p.d == 64 ? launch_logit<64>(p, L, st) : launch_logit<128>(p, L, st);
}

int launch_naive_attend_tc(const Problem& p, const void* A, cudaStream_t st) {
    return p.d == 64 ? launch_attend<64>(p, A, st) : launch_attend<128>(p, A, st);
}

}  // namespace flat

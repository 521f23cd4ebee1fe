// Fused Logit-Softmax-Attend on the sm_100a tensor cores (tcgen05 + TMEM + TMA), bf16 in,
// fp32 accumulate, bf16 out.
//
// Paper mapping (Section 5, 5.1, 5.2): the shared outer loops run over (batch, head) =
// blockIdx.y and the query-row tile = blockIdx.x (R-granularity, Rx = 128 rows).  The two
// inner loops -- Logit (S = Q K^T) and Attend (O += P V) -- run interleaved over 128-key
// tiles, with the softmax between them.  The paper's tile keeps all Nk logits of its rows
// on chip; one SM cannot (128 rows x 64K keys), so keys are streamed and the row maximum m
// and row sum l are carried along, which yields the same softmax exactly because
// sum_j e^{x_j - m'} = e^{m - m'} sum_j e^{x_j - m}.  Only Q, K, V are read from and O is
// written to device memory.
//
// Roles inside a CTA (192 threads):
//   warps 0-3  softmax: thread r owns query row r of the tile (TMEM lane r): reads its 128
//              logits from TMEM, keeps m and l in registers, writes bf16 weights P back to TMEM,
//              rescales O in TMEM when the reference maximum has to move, normalises and stores O;
//   warp 4     TMA producer (one lane): Q tile once, then K/V tiles into a 2-stage ring;
//   warp 5     MMA issuer (one lane): S = Q K^T into TMEM, then O += P V with P read from TMEM.
// Every wait is bounded: on expiry the kernel records a code in *status, raises a CTA-wide
// abort flag, drains its own copies, frees its TMEM and returns.
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

constexpr int BM = 128;              // query rows per CTA
constexpr int BN = 128;              // keys per step
constexpr int STAGES = 2;
constexpr int TC_THREADS = 192;
constexpr uint32_t TMEM_COLS = 256;

template <int D> struct TcLayout {
    static constexpr int Q_BYTES = BM * D * 2;
    static constexpr int KV_BYTES = BN * D * 2;
    static constexpr int TILE_BYTES = Q_BYTES + 2 * STAGES * KV_BYTES;
    static constexpr int SMEM_BYTES = TILE_BYTES + 256 + 1024;   // barriers + alignment slack
    static constexpr uint32_t S_COL = 0;
    static constexpr uint32_t O_COL = 128;
    static constexpr uint32_t P_COL = (D == 64) ? 192 : 0;       // d = 128: P overlays S columns 0..63
};

enum { BAR_Q_FULL = 0, BAR_KV_FULL = 1, BAR_KV_EMPTY = 1 + STAGES, BAR_S_FULL = 1 + 2 * STAGES,
       BAR_P_FULL, BAR_PV_DONE, NUM_BARS };

template <int D>
__global__ void __launch_bounds__(TC_THREADS, (D == 64) ? 2 : 1)
fused_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, int H, int Nq, int Nk,
                float scale_log2e, const int32_t* __restrict__ valid_len, int32_t* status) {
    using LY = TcLayout<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Qs = base;
    uint8_t* Ks = Qs + LY::Q_BYTES;                    // STAGES tiles
    uint8_t* Vs = Ks + STAGES * LY::KV_BYTES;          // STAGES tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + LY::TILE_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y;
    const int row0 = blockIdx.x * BM;
    int n = Nk;
    if (valid_len) { n = valid_len[bh / H]; n = n < 0 ? 0 : (n > Nk ? Nk : n); }
    const int ntiles = (n + BN - 1) / BN;

    if (threadIdx.x == 4 * 32) {
        mbar_init(&bars[BAR_Q_FULL], 1);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&bars[BAR_KV_FULL + s], 1); mbar_init(&bars[BAR_KV_EMPTY + s], 1); }
        mbar_init(&bars[BAR_S_FULL], 1);
        mbar_init(&bars[BAR_P_FULL], 128);
        mbar_init(&bars[BAR_PV_DONE], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0 && ntiles > 0) {
            prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
            mbar_arrive_expect_tx(&bars[BAR_Q_FULL], LY::Q_BYTES);
#pragma unroll
            for (int c = 0; c < D / 64; ++c) tma_load_3d(Qs + c * BM * 128, &tmQ, &bars[BAR_Q_FULL], c * 64, row0, bh);
            int issued = 0;
            bool ok = true;
            for (int j = 0; j < ntiles && ok; ++j) {
                const int s = j % STAGES;
                const uint32_t ph = (j / STAGES) & 1;
                ok = bounded_wait(&bars[BAR_KV_EMPTY + s], ph ^ 1, abort_flag, status, 0x100 + s);
                if (!ok) break;
                mbar_arrive_expect_tx(&bars[BAR_KV_FULL + s], 2 * LY::KV_BYTES);
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    tma_load_3d(Ks + s * LY::KV_BYTES + c * BN * 128, &tmK, &bars[BAR_KV_FULL + s], c * 64, j * BN, bh);
                    tma_load_3d(Vs + s * LY::KV_BYTES + c * BN * 128, &tmV, &bars[BAR_KV_FULL + s], c * 64, j * BN, bh);
                }
                issued = j + 1;
            }
            if (!ok) {
                // drain: wait (bounded) for the copies this thread started and nobody will consume
                drain_wait(&bars[BAR_Q_FULL], 0);
                for (int j = issued > STAGES ? issued - STAGES : 0; j < issued; ++j)
                    drain_wait(&bars[BAR_KV_FULL + j % STAGES], (j / STAGES) & 1);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && ntiles > 0) {
            constexpr uint32_t IDESC_S = make_idesc_bf16(BM, BN, 0, 0);
            constexpr uint32_t IDESC_PV = make_idesc_bf16(BM, D, 0, 1);
            bool ok = bounded_wait(&bars[BAR_Q_FULL], 0, abort_flag, status, 0x200);
            for (int j = 0; j < ntiles && ok; ++j) {
                const int s = j % STAGES;
                const uint32_t ph = (j / STAGES) & 1;
                ok = bounded_wait(&bars[BAR_KV_FULL + s], ph, abort_flag, status, 0x210 + s);
                if (!ok) break;
                tc_fence_after();
                const uint32_t q_addr = smem_u32(Qs), k_addr = smem_u32(Ks + s * LY::KV_BYTES),
                               v_addr = smem_u32(Vs + s * LY::KV_BYTES);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * (BM * 128) + (k % 4) * 32;
                    mma_ss(tmem + LY::S_COL, make_smem_desc_sw128(q_addr + off, 16, 1024),
                           make_smem_desc_sw128(k_addr + off, 16, 1024), IDESC_S, k > 0);
                }
                tc_commit(&bars[BAR_S_FULL]);
                ok = bounded_wait(&bars[BAR_P_FULL], j & 1, abort_flag, status, 0x220);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < BN / 16; ++k) {
                    mma_ts(tmem + LY::O_COL, tmem + LY::P_COL + k * 8,
                           make_smem_desc_sw128(v_addr + k * 2048, BN * 128, 1024), IDESC_PV, (j > 0 || k > 0));
                }
                tc_commit(&bars[BAR_KV_EMPTY + s]);
                tc_commit(&bars[BAR_PV_DONE]);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + epilogue (warps 0-3)
        const int row = row0 + warp * 32 + lane;
        const uint32_t tl = tmem + (static_cast<uint32_t>(warp * 32) << 16);
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < ntiles; ++j) {
            ok = bounded_wait(&bars[BAR_S_FULL], j & 1, abort_flag, status, 0x300);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int col0 = j * BN;
            const bool tail = col0 + BN > n;
            // pass 1: row maximum of the scaled logits
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tl + LY::S_COL + c * 32, r);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float x = __uint_as_float(r[i]) * scale_log2e;
                    if (tail && col0 + c * 32 + i >= n) x = -INFINITY;
                    mx = fmaxf(mx, x);
                }
            }
            if (__any_sync(0xffffffffu, mx > m_ref + RESCALE_THRESHOLD)) {
                const float m_new = fmaxf(m_ref, mx);
                const float alpha = ex2_approx(m_ref - m_new);     // 0 on the first tile
                l *= alpha;
                if (j > 0) {
                    ok = bounded_wait(&bars[BAR_PV_DONE], (j - 1) & 1, abort_flag, status, 0x310);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(tl + LY::O_COL + c * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st_x32(tl + LY::O_COL + c * 32, r);
                    }
                }
                m_ref = m_new;
            }
            // pass 2: p = 2^(x - m_ref), row sum in fp32 from the unrounded p, P rounded to bf16
            const float neg_m = -m_ref;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32], pk[16];
                tmem_ld_x32(tl + LY::S_COL + c * 32, r);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float x = fmaf(__uint_as_float(r[i]), scale_log2e, neg_m);
                    if (tail && col0 + c * 32 + i >= n) x = -INFINITY;
                    const float p = ex2_approx(x);
                    l += p;
                    r[i] = __float_as_uint(p);
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                tmem_st_x16(tl + LY::P_COL + c * 16, pk);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(&bars[BAR_P_FULL]);
        }
        if (ok && ntiles > 0) {
            ok = bounded_wait(&bars[BAR_PV_DONE], (ntiles - 1) & 1, abort_flag, status, 0x320);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            const float inv = l > 0.f ? 1.f / l : 0.f;
            tc_fence_after();
            __nv_bfloat16* orow = O + (static_cast<int64_t>(bh) * Nq + row) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                if (ntiles > 0) {
                    tmem_ld_x32(tl + LY::O_COL + c * 32, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;      // no valid key: O = 0
                }
                if (row < Nq) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(r[8 * v + 0]) * inv, __uint_as_float(r[8 * v + 1]) * inv);
                        w.y = pack_bf16x2(__uint_as_float(r[8 * v + 2]) * inv, __uint_as_float(r[8 * v + 3]) * inv);
                        w.z = pack_bf16x2(__uint_as_float(r[8 * v + 4]) * inv, __uint_as_float(r[8 * v + 5]) * inv);
                        w.w = pack_bf16x2(__uint_as_float(r[8 * v + 6]) * inv, __uint_as_float(r[8 * v + 7]) * inv);
                        *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = w;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// ---------------------------------------------------------------- host side
template <int D>
int launch_tc_d(const Problem& p, cudaStream_t st) {
    using LY = TcLayout<D>;
    CUtensorMap tmQ, tmK, tmV;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, D, BM) || !make_map(&tmK, p.K, BH, p.Nk, D, BN) ||
        !make_map(&tmV, p.V, BH, p.Nk, D, BN))
        return FLAT_ERR_CUDA;
    auto kern = fused_tc_kernel<D>;
    if (!ensure_dynamic_smem<fused_tc_kernel<D>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
    dim3 grid((p.Nq + BM - 1) / BM, BH);
    kern<<<grid, TC_THREADS, LY::SMEM_BYTES, st>>>(tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk,
                                                   p.scale * 1.4426950408889634f, p.k_valid_len, p.status);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

}  // namespace

int launch_fused_tc(const Problem& p, cudaStream_t st) {
    if (p.dtype != FLAT_DTYPE_BF16) return FLAT_ERR_UNSUPPORTED;
    if (p.d == 64) return launch_tc_d<64>(p, st);
    if (p.d == 128) return launch_tc_d<128>(p, st);
    return FLAT_ERR_UNSUPPORTED;
}

}  // namespace flat

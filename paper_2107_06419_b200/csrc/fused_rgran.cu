// The paper's row-granularity dataflow taken literally (Section 5.2, Fig. 7(b), and the buffer
// model of Section 5.3): a tile of R = 128 query rows keeps its WHOLE row of logits on chip --
// S = Q K^T for all keys at once -- the softmax then runs over complete rows in two passes (row
// maximum, then exponentials and row sum; no running maximum, nothing is ever rescaled), and
// O = P V follows.  On B200 the on-chip buffer for the R x N logits is TMEM (128 lanes x 512 fp32
// columns), so this form exists for up to 512 keys at d = 64 (bf16 in, fp32 accumulate, bf16 out);
// longer key sequences take the streaming kernels (fused_tc2.cu, fused_tc3.cu), which compute the
// same result.  It is the natural kernel for the shortest workload (512 x 512 per head): one pass,
// no ring buffers, every K and V tile resident in shared memory.
//
// CTA = 576 threads for one 128-row query tile:
//   warps 0-15  softmax: warp w serves rows 32 (w % 4) .. +31 (its TMEM lane quarter) and the key
//               tile w / 4 (128 keys, 128 logits per thread)
//   warp  16    TMA producer (one lane): Q, then all K tiles, then all V tiles, each on a barrier
//   warp  17    MMA issuer (one elected lane): S tile by tile as the K tiles land, then O = P V
// TMEM columns: S tile j at 128 j.  The weights P (bf16, two per column) of tile j are written over
// the first 64 columns of that tile by the threads that read them; once every weight is written the
// columns 64..127 of tile 0 are free and take the accumulator O.
// The four warps of a lane quarter exchange row maxima and row sums through shared memory around a
// named barrier of their 128 threads.  Every mbarrier wait is bounded (tc_common.cuh); a warp whose
// wait failed keeps going through all named barriers without doing work, so nothing hangs.
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

constexpr int RM = 128;              // query rows per CTA (the paper's R)
constexpr int RN = 128;              // keys per logit tile
constexpr int RD = 64;               // head size
constexpr int MAXT = 4;              // key tiles that fit TMEM: 4 x 128 fp32 columns
constexpr int RTHREADS = 32 * 16 + 64;

struct RL {
    static constexpr int TILE = RM * RD * 2;             // bytes of one 128 x 64 bf16 tile (Q, K_j or V_j)
    static constexpr int TILE_BYTES = (1 + 2 * MAXT) * TILE;
    static constexpr int XCH_BYTES = 2 * MAXT * RM * 4;  // [maximum | row sum][key tile][row]
    static constexpr int SMEM_BYTES = TILE_BYTES + XCH_BYTES + 256 + 1024;
    // barriers: Q, K[MAXT], V[MAXT], S_FULL[MAXT], P_FULL, O_FULL
    static constexpr int Q_FULL = 0, K_FULL = 1, V_FULL = K_FULL + MAXT, S_FULL = V_FULL + MAXT;
    static constexpr int P_FULL = S_FULL + MAXT, O_FULL = P_FULL + 1, NUM_BARS = O_FULL + 1;
    static constexpr uint32_t O_COL = 64;
};

__device__ __forceinline__ void quarter_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

__global__ void __launch_bounds__(RTHREADS, 1)
fused_rgran_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, int H, int Nq, int Nk,
                   float scale_log2e, const int32_t* __restrict__ valid_len, int coff, int32_t* status) {
    using LY = RL;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Qs = base;
    uint8_t* Ks = Qs + LY::TILE;
    uint8_t* Vs = Ks + MAXT * LY::TILE;
    float* xch = reinterpret_cast<float*>(base + LY::TILE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + LY::TILE_BYTES + LY::XCH_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + LY::NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y, row0 = blockIdx.x * RM;

    int n = Nk;
    if (valid_len) { n = valid_len[bh / H]; n = n < 0 ? 0 : (n > Nk ? Nk : n); }
    {
        // causal mask (coff = Nk - Nq; 2^30 = none): the tile's last row bounds the keys of all its rows
        const long long lim = static_cast<long long>(row0) + RM + coff;
        if (lim < n) n = lim < 0 ? 0 : static_cast<int>(lim);
    }
    const int ntiles = (n + RN - 1) / RN;                // <= MAXT (checked by the launcher)

    if (threadIdx.x == 16 * 32) {
        for (int i = 0; i < LY::NUM_BARS; ++i) mbar_init(&bars[i], i == LY::P_FULL ? 16 : 1);   // every softmax warp arrives once
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 16) {
        // ------------------------------------------------------------ TMA producer: everything at once
        if (lane == 0 && ntiles > 0) {
            prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
            mbar_arrive_expect_tx(&bars[LY::Q_FULL], LY::TILE);
            tma_load_3d(Qs, &tmQ, &bars[LY::Q_FULL], 0, row0, bh);
            for (int j = 0; j < ntiles; ++j) {
                mbar_arrive_expect_tx(&bars[LY::K_FULL + j], LY::TILE);
                tma_load_3d(Ks + j * LY::TILE, &tmK, &bars[LY::K_FULL + j], 0, j * RN, bh);
            }
            for (int j = 0; j < ntiles; ++j) {
                mbar_arrive_expect_tx(&bars[LY::V_FULL + j], LY::TILE);
                tma_load_3d(Vs + j * LY::TILE, &tmV, &bars[LY::V_FULL + j], 0, j * RN, bh);
            }
            // (this lane started the copies: it stays until they have landed, with a limit)
            drain_wait(&bars[LY::Q_FULL], 0);
            for (int j = 0; j < ntiles; ++j) { drain_wait(&bars[LY::K_FULL + j], 0); drain_wait(&bars[LY::V_FULL + j], 0); }
        }
    } else if (warp == 17) {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t IDESC_S = make_idesc_bf16(RM, RN, 0, 0);
        constexpr uint32_t IDESC_PV = make_idesc_bf16(RM, RD, 0, 1);
        const uint64_t q_desc = make_smem_desc_sw128(smem_u32(Qs), 16, 1024);
        const uint64_t k_desc = make_smem_desc_sw128(smem_u32(Ks), 16, 1024);
        const uint64_t v_desc = make_smem_desc_sw128(smem_u32(Vs), RN * 128, 1024);
        bool ok = true;
        auto wait = [&](int bar, int code) {
            if (ok) ok = __all_sync(0xffffffffu, bounded_wait(&bars[bar], 0, abort_flag, status, code));
            if (ok) tc_fence_after();
        };
        if (ntiles > 0) wait(LY::Q_FULL, 0x600);
        for (int j = 0; j < ntiles && ok; ++j) {
            wait(LY::K_FULL + j, 0x601);
            if (!ok) break;
            if (elect_one()) {
                const uint64_t kd = k_desc + static_cast<uint64_t>((j * LY::TILE) >> 4);
#pragma unroll
                for (int k = 0; k < RD / 16; ++k)
                    mma_ss(tmem + j * RN, q_desc + static_cast<uint64_t>((k * 32) >> 4),
                           kd + static_cast<uint64_t>((k * 32) >> 4), IDESC_S, k > 0);
                tc_commit(&bars[LY::S_FULL + j]);
            }
            __syncwarp();
        }
        if (ntiles > 0) wait(LY::P_FULL, 0x602);
        for (int j = 0; j < ntiles && ok; ++j) {
            wait(LY::V_FULL + j, 0x603);
            if (!ok) break;
            if (elect_one()) {
                const uint64_t vd = v_desc + static_cast<uint64_t>((j * LY::TILE) >> 4);
#pragma unroll
                for (int k = 0; k < RN / 16; ++k)
                    mma_ts(tmem + LY::O_COL, tmem + j * RN + k * 8, vd + static_cast<uint64_t>((k * 2048) >> 4),
                           IDESC_PV, (j > 0 || k > 0));
                if (j == ntiles - 1) tc_commit(&bars[LY::O_FULL]);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------ softmax (warps 0-15)
        const int q = warp & 3, kt = warp >> 2;
        const uint32_t tl = tmem + (static_cast<uint32_t>(q * 32) << 16);
        const int rloc = q * 32 + lane, row = row0 + rloc;
        const long long rlim = static_cast<long long>(row) + 1 + coff;
        const int nrow = rlim < n ? (rlim < 0 ? 0 : static_cast<int>(rlim)) : n;     // keys this row sees
        const int col0 = kt * RN;
        const int nvalid = nrow > col0 ? (nrow - col0 < RN ? nrow - col0 : RN) : 0;  // ... of this thread's key tile
        const bool active = kt < ntiles;
        bool ok = true;
        // ---- pass 1: the row maximum of x = scale * log2(e) * s over this thread's 128 logits
        float mx = -INFINITY;
        if (active) {
            ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::S_FULL + kt], 0, abort_flag, status, 0x610));
            tc_fence_after();
            if (ok) {
#pragma unroll
                for (int c = 0; c < RN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(tl + col0 + c * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c * 32 + i < nvalid) mx = fmaxf(mx, __uint_as_float(r[i]) * scale_log2e);
                }
            }
        }
        xch[kt * RM + rloc] = mx;
        quarter_sync(1 + q);
        float m = xch[rloc];
#pragma unroll
        for (int j = 1; j < MAXT; ++j) m = fmaxf(m, xch[j * RM + rloc]);
        // ---- pass 2: p = 2^(x - m), row sum, weights to TMEM over the first half of the logits just read
        float l = 0.f;
        if (active && ok) {
            const float neg_m = m == -INFINITY ? 0.f : -m;               // (a row without keys: every p is masked to 0)
#pragma unroll
            for (int c = 0; c < RN / 32; ++c) {
                uint32_t r[32], pk[16];
                tmem_ld_x32(tl + col0 + c * 32, r);
                tc_wait_ld();
                float p[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) p[i] = fmaf(__uint_as_float(r[i]), scale_log2e, neg_m);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    p[i] = ex2_approx(p[i]);
                    if (c * 32 + i >= nvalid) p[i] = 0.f;
                }
                float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    l0 += p[i]; l1 += p[i + 1]; l2 += p[i + 2]; l3 += p[i + 3];
                    pk[i / 2] = pack_bf16x2(p[i], p[i + 1]);
                    pk[i / 2 + 1] = pack_bf16x2(p[i + 2], p[i + 3]);
                }
                l += (l0 + l1) + (l2 + l3);
                tmem_st_x16(tl + col0 + c * 16, pk);
            }
            tc_wait_st();
        }
        xch[MAXT * RM + kt * RM + rloc] = l;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars[LY::P_FULL]);
        quarter_sync(1 + q);
        l = 0.f;
#pragma unroll
        for (int j = 0; j < MAXT; ++j) l += xch[MAXT * RM + j * RM + rloc];
        // ---- epilogue: this warp writes columns 16 kt .. 16 kt + 15 of its 32 rows
        if (ntiles > 0) ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::O_FULL], 0, abort_flag, status, 0x620)) && ok;
        if (ok) {
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            uint32_t r[16];
            if (ntiles > 0) {
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                    : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                      "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                    : "r"(tl + LY::O_COL + kt * 16)
                    : "memory");
                tc_wait_ld();
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) r[i] = 0u;
            }
            if (row < Nq) {
                __nv_bfloat16* orow = O + (static_cast<int64_t>(bh) * Nq + row) * RD + kt * 16;
                uint4 w0, w1;
                w0.x = pack_bf16x2(__uint_as_float(r[0]) * inv, __uint_as_float(r[1]) * inv);
                w0.y = pack_bf16x2(__uint_as_float(r[2]) * inv, __uint_as_float(r[3]) * inv);
                w0.z = pack_bf16x2(__uint_as_float(r[4]) * inv, __uint_as_float(r[5]) * inv);
                w0.w = pack_bf16x2(__uint_as_float(r[6]) * inv, __uint_as_float(r[7]) * inv);
                w1.x = pack_bf16x2(__uint_as_float(r[8]) * inv, __uint_as_float(r[9]) * inv);
                w1.y = pack_bf16x2(__uint_as_float(r[10]) * inv, __uint_as_float(r[11]) * inv);
                w1.z = pack_bf16x2(__uint_as_float(r[12]) * inv, __uint_as_float(r[13]) * inv);
                w1.w = pack_bf16x2(__uint_as_float(r[14]) * inv, __uint_as_float(r[15]) * inv);
                *reinterpret_cast<uint4*>(orow) = w0;
                *reinterpret_cast<uint4*>(orow + 8) = w1;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace

bool rgran_applies(const Problem& p) {
    return p.dtype == FLAT_DTYPE_BF16 && p.d == RD && p.Nk <= MAXT * RN;
}

int launch_fused_rgran(const Problem& p, cudaStream_t st) {
    if (!rgran_applies(p)) return FLAT_ERR_UNSUPPORTED;
    using LY = RL;
    CUtensorMap tmQ, tmK, tmV;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, RD, RM) || !make_map(&tmK, p.K, BH, p.Nk, RD, RN) ||
        !make_map(&tmV, p.V, BH, p.Nk, RD, RN))
        return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<fused_rgran_kernel>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
    dim3 grid((p.Nq + RM - 1) / RM, BH);
    fused_rgran_kernel<<<grid, RTHREADS, LY::SMEM_BYTES, st>>>(tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq,
                                                               p.Nk, p.scale * 1.4426950408889634f, p.k_valid_len,
                                                               p.causal ? p.Nk - p.Nq : (1 << 30), p.status);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

}  // namespace flat

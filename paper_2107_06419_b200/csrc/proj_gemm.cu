// The activation-weight operators of an attention layer (Section 2, "Computation operators",
// steps 1 and 5): the Query / Key / Value projections of the input [B,N,D] into [B,H,N,d] and the
// Output projection of the concatenated heads back to [B,N,D].  Both are Y = A W^T with bf16
// operands, fp32 accumulation in TMEM and bf16 results, as one persistent tcgen05 kernel:
//   * the Q/K/V projection is ONE contraction against the stacked weights [3 H d, D]; its epilogue
//     writes each output tile straight into the head-major tensors Q, K, V [B,H,N,d] that the
//     fused attention kernel reads (no transposition pass);
//   * the Output projection reads its A operand straight from the head-major attention output
//     O [B,H,N,d]: a 64-wide slice of the contraction index h * d + c is a (head, column) box of
//     that tensor for TMA.
// CTA = 320 threads: warps 0-7 epilogue (TMEM -> bf16 -> global), warp 8 TMA producer (one lane),
// warp 9 MMA issuer (one elected lane).  Tiles of 256 x 256 outputs as two row blocks of 128 that
// share every 256-row tile of W (each W byte fetched feeds twice the MMAs); contraction in slices
// of 64 through a three-stage ring (64 KB per stage); the two accumulators fill TMEM (2 x 256
// columns), so a tile's epilogue is not overlapped with the next tile's MMAs (about a tenth of a
// tile's time at a contraction length of 1024; tiles of 128 x 256 with two alternating
// accumulators, which do overlap it, measured 1.6 % slower).  A CTA walks tiles blockIdx.x,
// blockIdx.x + gridDim.x, ...; tiles that share their rows of A are neighbours, so CTAs running
// together share A in L2 (the weights fit L2 whole).  Every wait is bounded (tc_common.cuh).
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

constexpr int GM = 256;              // output rows per tile: two MMA row blocks of 128 that share the W tile
constexpr int GN = 256;              // output columns per tile
constexpr int GK = 64;               // contraction slice (one 128-byte swizzle atom of bf16)
constexpr int STAGES = 3;
constexpr int GTHREADS = 320;        // 8 epilogue warps, TMA producer, MMA issuer

struct GL {
    static constexpr int A_BYTES = GM * GK * 2;
    static constexpr int B_BYTES = GN * GK * 2;
    static constexpr int TILE_BYTES = STAGES * (A_BYTES + B_BYTES);
    static constexpr int SMEM_BYTES = TILE_BYTES + 256 + 1024;
    static constexpr uint32_t TMEM_COLS = 512;           // the accumulators of the two row blocks, GN columns each
    // barriers: FULL[STAGES], EMPTY[STAGES], ACC_FULL, ACC_EMPTY
    static constexpr int FULL = 0, EMPTY = STAGES, ACC_FULL = 2 * STAGES, ACC_EMPTY = ACC_FULL + 1;
    static constexpr int NUM_BARS = ACC_EMPTY + 1;
};

struct GemmArgs {
    int M, Nout, Kdim;               // Y [M, Nout] = A [M, Kdim] W[Nout, Kdim]^T
    int N, H, d;                     // tokens per sequence, heads, head size (head-major sides)
    __nv_bfloat16* out0;             // token-major Y, or head-major Q
    __nv_bfloat16* out1;             // head-major K
    __nv_bfloat16* out2;             // head-major V
    int wide_stores;                 // every output pointer is 32-byte aligned: 32-byte stores
};

// A_HEADS: A is the head-major tensor [B,H,N,d] (Output projection); else token-major [M, Kdim].
// OUT_HEADS: the result goes to the head-major tensors out0..2 (Q/K/V projection); else to the
// token-major Y = out0.
template <bool A_HEADS, bool OUT_HEADS>
__global__ void __launch_bounds__(GTHREADS, 1)
proj_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, const GemmArgs g,
                 int32_t* status) {
    using LY = GL;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* As = base;
    uint8_t* Bs = base + STAGES * LY::A_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + LY::TILE_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + LY::NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 8 * 32) {
        for (int i = 0; i < LY::NUM_BARS; ++i) mbar_init(&bars[i], i >= LY::ACC_EMPTY ? 8 : 1);   // eight epilogue warps free the accumulators
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, LY::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int tiles_n = g.Nout / GN, tiles_m = (g.M + GM - 1) / GM;
    const int tiles = tiles_m * tiles_n, ksteps = g.Kdim / GK;

    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tmA); prefetch_tensormap(&tmW);
            bool ok = true;
            int issued = 0, it = 0;                      // it: ring slot counter over all tiles
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int m0 = (tile / tiles_n) * GM, n0 = (tile % tiles_n) * GN;
                for (int kc = 0; kc < ksteps && ok; ++kc, ++it) {
                    const int s = it % STAGES;
                    ok = bounded_wait(&bars[LY::EMPTY + s], ((it / STAGES) & 1) ^ 1, abort_flag, status, 0x500);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&bars[LY::FULL + s], LY::A_BYTES + LY::B_BYTES);
                    if (A_HEADS) {
                        // each block of 128 rows holds tokens of ONE sequence (N is a multiple of 128); slice
                        // kc of the contraction index h * d + c lies in one head.  (A block past the last
                        // sequence has an out-of-range coordinate and reads zeros.)
                        const int k0 = kc * GK, h = k0 / g.d, c0 = k0 - h * g.d;
#pragma unroll
                        for (int r = 0; r < GM / 128; ++r) {
                            const int mr = m0 + r * 128, b = mr / g.N, tok0 = mr - b * g.N;
                            tma_load_3d(As + s * LY::A_BYTES + r * 128 * GK * 2, &tmA, &bars[LY::FULL + s], c0, tok0,
                                        b * g.H + h);
                        }
                    } else {
#pragma unroll
                        for (int r = 0; r < GM / 128; ++r)
                            tma_load_3d(As + s * LY::A_BYTES + r * 128 * GK * 2, &tmA, &bars[LY::FULL + s], kc * GK,
                                        m0 + r * 128, 0);
                    }
                    tma_load_3d(Bs + s * LY::B_BYTES, &tmW, &bars[LY::FULL + s], kc * GK, n0, 0);
                    issued = it + 1;
                }
            }
            if (!ok)
                for (int j = issued > STAGES ? issued - STAGES : 0; j < issued; ++j)
                    drain_wait(&bars[LY::FULL + j % STAGES], (j / STAGES) & 1);
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer
        constexpr uint32_t IDESC = make_idesc_bf16(128, GN, 0, 0);
        const uint64_t ad = make_smem_desc_sw128(smem_u32(As), 16, 1024);
        const uint64_t bd = make_smem_desc_sw128(smem_u32(Bs), 16, 1024);
        bool ok = true;
        int it = 0, tcount = 0;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
            // the epilogue must have read the accumulators of the previous tile
            if (tcount >= 1)
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::ACC_EMPTY], (tcount - 1) & 1, abort_flag,
                                                          status, 0x510));
            if (!ok) break;
            tc_fence_after();
            for (int kc = 0; kc < ksteps && ok; ++kc, ++it) {
                const int s = it % STAGES;
                ok = __all_sync(0xffffffffu,
                                bounded_wait(&bars[LY::FULL + s], (it / STAGES) & 1, abort_flag, status, 0x520));
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t a = ad + static_cast<uint64_t>((s * LY::A_BYTES) >> 4);
                    const uint64_t b = bd + static_cast<uint64_t>((s * LY::B_BYTES) >> 4);
#pragma unroll
                    for (int k = 0; k < GK / 16; ++k)
#pragma unroll
                        for (int r = 0; r < GM / 128; ++r)
                            mma_ss(tmem + r * GN, a + static_cast<uint64_t>((r * 128 * GK * 2 + k * 32) >> 4),
                                   b + static_cast<uint64_t>((k * 32) >> 4), IDESC, (kc > 0 || k > 0));
                    tc_commit(&bars[LY::EMPTY + s]);
                    if (kc == ksteps - 1) tc_commit(&bars[LY::ACC_FULL]);
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 0-7)
        // warp w reads TMEM lanes 32 (w % 4) .. of row block w / 4
        bool ok = true;
        int tcount = 0;
        const int rb = warp >> 2;
        const uint32_t tl = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16) + rb * GN;
        const int HD = g.H * g.d;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
            const int m0 = (tile / tiles_n) * GM, n0 = (tile % tiles_n) * GN;
            const int m = m0 + warp * 32 + lane;
            ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::ACC_FULL], tcount & 1, abort_flag, status, 0x530));
            if (!ok) break;
            tc_fence_after();
            int64_t row_off = 0;                         // element offset of this thread's row in its destination
            int b = 0, tok = 0;
            if (OUT_HEADS) { b = m / g.N; tok = m - b * g.N; }
            else row_off = static_cast<int64_t>(m) * g.Nout + n0;
            // First the whole accumulator row goes to registers as packed bf16 (128 words), so that the
            // accumulator is released for the next tile's MMAs before any store is issued.
            uint32_t w[GN / 2];
#pragma unroll
            for (int c = 0; c < GN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tl + c * 32, r);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    w[c * 16 + i] = pack_bf16x2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[LY::ACC_EMPTY]);
            if (m < g.M) {
#pragma unroll
                for (int c = 0; c < GN / 32; ++c) {
                    __nv_bfloat16* dst;
                    if (OUT_HEADS) {
                        // 32 consecutive output columns lie in one head of one of Q, K, V (32 divides d)
                        const int n = n0 + c * 32, which = n / HD, rem = n - which * HD, h = rem / g.d, cc = rem - h * g.d;
                        __nv_bfloat16* o = which == 0 ? g.out0 : (which == 1 ? g.out1 : g.out2);
                        dst = o + ((static_cast<int64_t>(b) * g.H + h) * g.N + tok) * g.d + cc;
                    } else {
                        dst = g.out0 + row_off + c * 32;
                    }
                    if (g.wide_stores) {
                        st_global_32B(dst, *reinterpret_cast<uint32_t(*)[8]>(&w[c * 16]));
                        st_global_32B(dst + 16, *reinterpret_cast<uint32_t(*)[8]>(&w[c * 16 + 8]));
                    } else {
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            *reinterpret_cast<uint4*>(dst + v * 8) =
                                make_uint4(w[c * 16 + 4 * v], w[c * 16 + 4 * v + 1], w[c * 16 + 4 * v + 2], w[c * 16 + 4 * v + 3]);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, LY::TMEM_COLS);
}

// [rows, cols] bf16 row-major as a TMA tensor with boxes of 64 columns x box_rows rows.
bool make_map_2d(CUtensorMap* m, const void* ptr, int rows, int cols, int box_rows) {
    return make_map(m, ptr, 1, rows, cols, box_rows);
}

template <bool A_HEADS, bool OUT_HEADS>
int launch_gemm(const CUtensorMap& tmA, const CUtensorMap& tmW, const GemmArgs& g, int32_t* status, cudaStream_t st) {
    if (!ensure_dynamic_smem<proj_gemm_kernel<A_HEADS, OUT_HEADS>>(GL::SMEM_BYTES)) return FLAT_ERR_CUDA;
    const int tiles = ((g.M + GM - 1) / GM) * (g.Nout / GN);
    const int sms = device_sm_count();
    const int grid = tiles < sms ? tiles : sms;
    proj_gemm_kernel<A_HEADS, OUT_HEADS><<<grid, GTHREADS, GL::SMEM_BYTES, st>>>(tmA, tmW, g, status);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31) == 0; }

}  // namespace

int launch_qkv_proj(const void* X, const void* Wqkv, void* Q, void* K, void* V, int B, int N, int H, int d, int Dm,
                    int32_t* status, cudaStream_t st) {
    if (!X || !Wqkv || !Q || !K || !V) return FLAT_ERR_NULL;
    if (B < 1 || N < 1 || H < 1 || Dm < 1) return FLAT_ERR_SHAPE;
    if (static_cast<int64_t>(B) * N > 0x7fffffff || static_cast<int64_t>(H) * d * 3 > 0x7fffffff) return FLAT_ERR_SHAPE;
    if ((d != 64 && d != 128) || (H * d) % GN != 0 || Dm % GK != 0) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(Wqkv) || !aligned16(Q) || !aligned16(K) || !aligned16(V)) return FLAT_ERR_ALIGN;
    GemmArgs g{B * N, 3 * H * d, Dm, N, H, d, static_cast<__nv_bfloat16*>(Q), static_cast<__nv_bfloat16*>(K),
               static_cast<__nv_bfloat16*>(V), aligned32(Q) && aligned32(K) && aligned32(V)};
    CUtensorMap tmA, tmW;
    if (!make_map_2d(&tmA, X, g.M, Dm, 128) || !make_map_2d(&tmW, Wqkv, g.Nout, Dm, GN)) return FLAT_ERR_CUDA;
    return launch_gemm<false, true>(tmA, tmW, g, status, st);
}

int launch_out_proj(const void* O, const void* Wo, void* Y, int B, int N, int H, int d, int Dm, int32_t* status,
                    cudaStream_t st) {
    if (!O || !Wo || !Y) return FLAT_ERR_NULL;
    if (B < 1 || N < 1 || H < 1 || Dm < 1) return FLAT_ERR_SHAPE;
    if (static_cast<int64_t>(B) * N > 0x7fffffff || static_cast<int64_t>(B) * H > 0x7fffffff) return FLAT_ERR_SHAPE;
    if ((d != 64 && d != 128) || N % 128 != 0 || Dm % GN != 0) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(O) || !aligned16(Wo) || !aligned16(Y)) return FLAT_ERR_ALIGN;
    GemmArgs g{B * N, Dm, H * d, N, H, d, static_cast<__nv_bfloat16*>(Y), nullptr, nullptr, aligned32(Y)};
    CUtensorMap tmA, tmW;
    if (!make_map(&tmA, O, B * H, N, d, 128) || !make_map_2d(&tmW, Wo, Dm, H * d, GN)) return FLAT_ERR_CUDA;
    return launch_gemm<true, false>(tmA, tmW, g, status, st);
}

int launch_fc(const void* X, const void* W, void* Y, int M, int Kdim, int Nout, int32_t* status, cudaStream_t st) {
    if (!X || !W || !Y) return FLAT_ERR_NULL;
    if (M < 1 || Kdim < 1 || Nout < 1) return FLAT_ERR_SHAPE;
    if (Kdim % GK != 0 || Nout % GN != 0) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(W) || !aligned16(Y)) return FLAT_ERR_ALIGN;
    GemmArgs g{M, Nout, Kdim, M, 1, 64, static_cast<__nv_bfloat16*>(Y), nullptr, nullptr, aligned32(Y)};
    CUtensorMap tmA, tmW;
    if (!make_map_2d(&tmA, X, M, Kdim, 128) || !make_map_2d(&tmW, W, Nout, Kdim, GN)) return FLAT_ERR_CUDA;
    return launch_gemm<false, false>(tmA, tmW, g, status, st);
}

}  // namespace flat

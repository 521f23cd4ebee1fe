// Backward pass of the fused Logit-softmax-Attend on the sm_100a tensor cores (tcgen05 + TMEM + TMA):
// bf16 in, fp32 accumulate, bf16 gradients out.
//
// The paper stops at inference; this is the chain rule on its Section 2 steps 2-4, computed with the
// same idea as its Section 5 dataflow: the [Nq, Nk] intermediates (weights P, their gradient dP and the
// logit gradient dS) are rebuilt tile by tile on chip and never reach device memory.  With S = scale Q K^T,
// lse the row-wise log-sum-exp that the forward pass saved, P = exp(S - lse) and delta_i = sum_t dO[i,t] O[i,t]:
//     dV = P^T dO        dP = dO V^T        dS = P o (dP - delta)        dQ = scale dS K        dK = scale dS^T Q
// Two launches of one kernel template, no atomics and no workspace beyond delta [B,H,Nq]:
//   MODE_DQ : one CTA per 128 query rows, streaming key tiles:   S = Q K^T, dP = dO V^T, dQ += dS K.
//             Also computes delta for its rows and writes it for the second launch.
//   MODE_DKV: one CTA per 128 keys, streaming query tiles:       S^T = K Q^T, dP^T = V dO^T,
//             dV += P^T dO, dK += dS^T Q.
// Both are the same program: a stationary pair of tiles (X1, X2) whose rows are the TMEM lanes, a streamed
// pair (Y1, Y2) whose rows are the columns:  T1 = X1 Y1^T,  T2 = X2 Y2^T  (both operands K-major in shared
// memory), then element-wise p = 2^(c T1 - lse2), ds = p (T2 - delta) with lse2 / delta taken per lane
// (MODE_DQ) or per column (MODE_DKV), P and dS rounded to bf16 and written back to TMEM, and
// acc_a += dS Y1, acc_b += P Y2 with the bf16 tile as the TMEM A-operand and Y as an MN-major B-operand.
//
// The streamed tile is worked on in two halves of 64 columns (a: rows 0-63 of Y, b: rows 64-127), each with
// its own 64 columns of T1 / T2, so that the MMAs of one half run under the element-wise work of the other.
// Where TMEM has room beside T1, T2 and the accumulators (every case but MODE_DKV at d = 128) the bf16 tiles
// get columns of their own, and the next step's T of a half is issued AHEAD of this step's accumulation
// (which only has to finish before the element-wise warps write the next bf16 tile: barrier ACC_HALF);
// otherwise P / dS overlay the T columns they were computed from and the accumulation goes first.
//
// CTA = 576 threads: warps 0-15 element-wise (warp w: TMEM lane quarter w % 4, half step w / 8, 32 of that
// half's 64 columns: (w / 4) % 2 -- four warps per scheduler, two of each half, so that the waits of one
// (barrier, TMEM load, store completion) hide behind the exponentials of the others), warp 16 TMA producer
// (and, in MODE_DKV, the per-column lse2 / delta vectors of every streamed tile, converted and put into
// shared memory), warp 17 MMA issuer.
// Every wait is bounded (tc_common.cuh); on expiry the CTA aborts cleanly and reports a code.
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

constexpr int BT = 128;              // rows of every tile (queries or keys)
constexpr int HC = 64;               // columns (rows of the streamed tile) per half step
constexpr int EW_WARPS = 16;           // eight per half step
constexpr int BWD_THREADS = 32 * EW_WARPS + 64;
constexpr int MODE_DQ = 0, MODE_DKV = 1;
constexpr float LOG2E = 1.4426950408889634f;

template <int D, int MODE> struct BL {
    static constexpr int TILE_BYTES = BT * D * 2;
    // Ring of streamed HALF tile pairs (64 rows of Y1 and of Y2 per stage, one stage per half step): deep
    // enough that a copy (about two microseconds from device memory) is under way for every half step the
    // element-wise warps and the MMAs are working on, and released half by half.
    static constexpr int HTILE_BYTES = HC * D * 2;
    static constexpr int HSTAGES = D == 64 ? 8 : 4;
    static constexpr int VSTAGES = HSTAGES / 2;                              // ring of per-column vectors (whole steps)
    static constexpr int OPERAND_BYTES = 2 * TILE_BYTES + 2 * HSTAGES * HTILE_BYTES;   // X1, X2, HSTAGES x (Y1, Y2 halves)
    static constexpr int VEC_BYTES = VSTAGES * 2 * BT * 4;                   // [stage][lse2 | delta][column]
    static constexpr int XCH_BYTES = 4 * BT * 4;                             // delta quarters of MODE_DQ
    static constexpr int SMEM_BYTES = OPERAND_BYTES + VEC_BYTES + XCH_BYTES + 512 + 1024;
    static constexpr uint32_t T1_COL = 0, T2_COL = 128, ACC_A_COL = 256, ACC_B_COL = 256 + D;
    static constexpr uint32_t ACC_END = 256 + (MODE == MODE_DKV ? 2 : 1) * D;
    static constexpr bool SEP = ACC_END + 128 <= 512;                        // room for the bf16 tiles beside T1 / T2
    static constexpr uint32_t DS_COL = ACC_END, P_COL = ACC_END + 64;        // (SEP) 32 columns per half each
    static constexpr uint32_t TMEM_COLS = 512;
    // columns of the bf16 dS / P tile that element-wise warp-half h (0 / 1) writes in half step `half`,
    // and of contraction slice k (16 indices, k = 0..3) of that half step
    __host__ __device__ static constexpr uint32_t ds_store(int half, int h) { return SEP ? DS_COL + half * 32 + h * 16 : T2_COL + half * HC + h * 32; }
    __host__ __device__ static constexpr uint32_t p_store(int half, int h) { return SEP ? P_COL + half * 32 + h * 16 : T1_COL + half * HC + h * 32; }
    __host__ __device__ static constexpr uint32_t ds_slice(int half, int k) { return ds_store(half, k / 2) + (k % 2) * 8; }
    __host__ __device__ static constexpr uint32_t p_slice(int half, int k) { return p_store(half, k / 2) + (k % 2) * 8; }
    // barriers.  T_FULL / PD_FULL / ACC_HALF [half]: the half's T1, T2 are computed / its dS (and P) are
    // written / the MMAs that read them have completed -- once per step each; VEC_FULL [stage]: the step's
    // lse2 / delta vectors are in shared memory (MODE_DKV)
    static constexpr int BAR_X_FULL = 0, BAR_Y_FULL = 1, BAR_Y_EMPTY = 1 + HSTAGES, BAR_T_FULL = 1 + 2 * HSTAGES,
                         BAR_PD_FULL = BAR_T_FULL + 2, BAR_ACC_HALF = BAR_PD_FULL + 2, BAR_VEC_FULL = BAR_ACC_HALF + 2,
                         BAR_ACC_DONE = BAR_VEC_FULL + VSTAGES, NUM_BARS = BAR_ACC_DONE + 1;
};

__device__ __forceinline__ void ew_sync() { asm volatile("bar.sync 1, 512;" ::: "memory"); }

// X1, X2 / Y1, Y2 by mode:  MODE_DQ: (Q, dO) / (K, V);  MODE_DKV: (K, V) / (Q, dO).
template <int D, int MODE>
__global__ void __launch_bounds__(BWD_THREADS, 1)
bwd_tc_kernel(const __grid_constant__ CUtensorMap tmX1, const __grid_constant__ CUtensorMap tmX2,
              const __grid_constant__ CUtensorMap tmY1, const __grid_constant__ CUtensorMap tmY2,
              const __nv_bfloat16* __restrict__ dOg, const __nv_bfloat16* __restrict__ Og,
              const float* __restrict__ lse, float* __restrict__ delta,
              __nv_bfloat16* __restrict__ outA, __nv_bfloat16* __restrict__ outB,
              int H, int Nq, int Nk, float scale, const int32_t* __restrict__ valid_len, int coff, int32_t* status) {
    using LY = BL<D, MODE>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* X1s = base;
    uint8_t* X2s = X1s + LY::TILE_BYTES;
    uint8_t* Ys = X2s + LY::TILE_BYTES;                  // half stage s: Y1 rows at 2 s, Y2 rows at 2 s + 1 (half tiles)
    float* vec = reinterpret_cast<float*>(base + LY::OPERAND_BYTES);
    float* xch = vec + LY::VSTAGES * 2 * BT;
    uint64_t* bars = reinterpret_cast<uint64_t*>(xch + 4 * BT);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + LY::NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y;
    const int x0 = blockIdx.x * BT;                      // first row of the stationary tile (query or key)
    const int NX = MODE == MODE_DQ ? Nq : Nk;            // rows of the stationary tensors
    int nkeys = Nk;                                      // keys of this batch that take part at all
    if (valid_len) { nkeys = valid_len[bh / H]; nkeys = nkeys < 0 ? 0 : (nkeys > Nk ? Nk : nkeys); }
    // Range of streamed tiles [y_begin, y_end) that hold at least one visible (query, key) pair.
    // Causal mask (coff = Nk - Nq; 2^30 = none): query i sees key j iff j <= i + coff.
    int y_begin = 0, y_end;
    if (MODE == MODE_DQ) {
        const long long lim = static_cast<long long>(x0) + BT + coff;          // keys below this for the tile's last row
        const int n = lim < nkeys ? (lim < 0 ? 0 : static_cast<int>(lim)) : nkeys;
        y_end = (n + BT - 1) / BT;
    } else {
        y_end = x0 < nkeys ? (Nq + BT - 1) / BT : 0;
        const long long first = static_cast<long long>(x0) - coff;             // first query that sees key x0
        if (first > 0) y_begin = static_cast<int>(first / BT < y_end ? first / BT : y_end);
    }
    const int nsteps = y_end - y_begin;

    if (threadIdx.x == EW_WARPS * 32) {
        for (int i = 0; i < LY::NUM_BARS; ++i) mbar_init(&bars[i], (i >= LY::BAR_PD_FULL && i < LY::BAR_ACC_HALF) ? EW_WARPS / 2 : 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, LY::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    auto wait_warp = [&](int bar, uint32_t parity, int code) {
        return __all_sync(0xffffffffu, bounded_wait(&bars[bar], parity, abort_flag, status, code));
    };

    if (warp == EW_WARPS) {
        // ------------------------------------------------------------ TMA producer (+ column vectors)
        // The whole warp walks the loop; lane 0 issues the copies.  MODE_DKV: the 32 lanes also fetch
        // the streamed tile's lse and delta (4 columns each), turn lse into base-2 units (+inf switches a
        // column off: a query without keys, or past the end) and put both into the step's buffer.
        if (nsteps > 0) {
            if (lane == 0) {
                prefetch_tensormap(&tmX1); prefetch_tensormap(&tmX2); prefetch_tensormap(&tmY1); prefetch_tensormap(&tmY2);
                mbar_arrive_expect_tx(&bars[LY::BAR_X_FULL], 2 * LY::TILE_BYTES);
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    tma_load_3d(X1s + c * BT * 128, &tmX1, &bars[LY::BAR_X_FULL], c * 64, x0, bh);
                    tma_load_3d(X2s + c * BT * 128, &tmX2, &bars[LY::BAR_X_FULL], c * 64, x0, bh);
                }
            }
            int issued = 0;
            bool ok = true;
            for (int g = 0; g < 2 * nsteps && ok; ++g) {     // half steps: g = 2 j + half
                const int s = g % LY::HSTAGES, j = g >> 1, half = g & 1;
                ok = wait_warp(LY::BAR_Y_EMPTY + s, ((g / LY::HSTAGES) & 1) ^ 1, 0x500 + s);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bars[LY::BAR_Y_FULL + s], 2 * LY::HTILE_BYTES);
#pragma unroll
                    for (int c = 0; c < D / 64; ++c) {
                        tma_load_3d(Ys + (2 * s) * LY::HTILE_BYTES + c * HC * 128, &tmY1, &bars[LY::BAR_Y_FULL + s], c * 64,
                                    (y_begin + j) * BT + half * HC, bh);
                        tma_load_3d(Ys + (2 * s + 1) * LY::HTILE_BYTES + c * HC * 128, &tmY2, &bars[LY::BAR_Y_FULL + s], c * 64,
                                    (y_begin + j) * BT + half * HC, bh);
                    }
                }
                issued = g + 1;
                if (MODE == MODE_DKV && half == 1) {
                    // The step's vectors go into ring slot j % VSTAGES, last read in step j - VSTAGES.  The
                    // stage just granted (the SECOND half's) was released behind the second half of that
                    // step, i.e. after all of its element-wise work.
                    float l2[4], dl[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i = (y_begin + j) * BT + lane * 4 + e;
                        l2[e] = INFINITY; dl[e] = 0.f;
                        if (i < Nq) {
                            const float l = lse[static_cast<int64_t>(bh) * Nq + i];
                            l2[e] = l == -INFINITY ? INFINITY : l * LOG2E;
                            dl[e] = delta[static_cast<int64_t>(bh) * Nq + i];
                        }
                    }
                    float* vb = vec + (j % LY::VSTAGES) * 2 * BT + lane * 4;
                    *reinterpret_cast<float4*>(vb) = make_float4(l2[0], l2[1], l2[2], l2[3]);
                    *reinterpret_cast<float4*>(vb + BT) = make_float4(dl[0], dl[1], dl[2], dl[3]);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars[LY::BAR_VEC_FULL + j % LY::VSTAGES]);
                }
            }
            if (!ok && lane == 0) {
                drain_wait(&bars[LY::BAR_X_FULL], 0);
                for (int g = issued > LY::HSTAGES ? issued - LY::HSTAGES : 0; g < issued; ++g)
                    drain_wait(&bars[LY::BAR_Y_FULL + g % LY::HSTAGES], (g / LY::HSTAGES) & 1);
            }
        }
    } else if (warp == EW_WARPS + 1) {
        // ------------------------------------------------------------ MMA issuer
        //   T(j, half):   T1 = X1 Y1[half]^T and T2 = X2 Y2[half]^T into the half's 64 columns of T1 / T2;
        //   ACC(j, half): once the element-wise warps have written the half's dS (and P):
        //                 acc_a += dS Y1[half] (and acc_b += P Y2[half]).
        // Issue order per half, behind PD_FULL(j, half):  T(j+1, half) then ACC(j, half) where the bf16
        // tiles have columns of their own; ACC(j, half) then T(j+1, half) where they overlay T1 / T2 (the
        // MMAs of one thread execute in issue order, so the T that overwrites them needs no wait).
        // The whole warp walks the loop (uniform control flow) and one elected lane issues: the MMA and
        // commit instructions take their operands from uniform registers, which the compiler can only
        // use when it knows that a single thread runs the code.
        if (nsteps > 0) {
            constexpr uint32_t IDESC_T = make_idesc_bf16(BT, HC, 0, 0);
            constexpr uint32_t IDESC_ACC = make_idesc_bf16(BT, D, 0, 1);
            bool ok = wait_warp(LY::BAR_X_FULL, 0, 0x510);
            // descriptors of the first feature slice of each operand (the others are constant offsets away)
            const uint64_t x1d = make_smem_desc_sw128(smem_u32(X1s), 16, 1024);            // K-major
            const uint64_t x2d = make_smem_desc_sw128(smem_u32(X2s), 16, 1024);
            const uint64_t ykd = make_smem_desc_sw128(smem_u32(Ys), 16, 1024);             // Y1 half of stage 0, K-major
            const uint64_t ymd = make_smem_desc_sw128(smem_u32(Ys), HC * 128, 1024);       // Y1 half of stage 0, MN-major
            constexpr uint64_t HTILE16 = LY::HTILE_BYTES >> 4;                              // descriptor units of 16 bytes
            // Consecutive MMAs into ONE accumulator wait for each other, so the slices of independent
            // products are issued in turn: T1 and T2 of a half, and the accumulations acc_a and acc_b.
            auto issue_t = [&](int j, int half) {
                // (feature slice k of a K-major operand: panel k / 4 of 64 features, 32 bytes per slice; a panel
                // is 128 rows of 128 bytes for the stationary tiles, 64 rows for the streamed half tiles)
                const uint64_t y1 = ykd + static_cast<uint64_t>(2 * ((2 * j + half) % LY::HSTAGES)) * HTILE16;
                const uint64_t y2 = y1 + HTILE16;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint64_t xoff = static_cast<uint64_t>(((k / 4) * (BT * 128) + (k % 4) * 32) >> 4);
                    const uint64_t yoff = static_cast<uint64_t>(((k / 4) * (HC * 128) + (k % 4) * 32) >> 4);
                    mma_ss(tmem + LY::T1_COL + half * HC, x1d + xoff, y1 + yoff, IDESC_T, k > 0);
                    mma_ss(tmem + LY::T2_COL + half * HC, x2d + xoff, y2 + yoff, IDESC_T, k > 0);
                }
                tc_commit(&bars[LY::BAR_T_FULL + half]);
            };
            auto issue_acc = [&](int j, int half) {
                const uint64_t y1 = ymd + static_cast<uint64_t>(2 * ((2 * j + half) % LY::HSTAGES)) * HTILE16;
                const uint64_t y2 = y1 + HTILE16;
                const uint32_t acc = (j > 0 || half > 0) ? 1u : 0u;
#pragma unroll
                for (int k = 0; k < HC / 16; ++k) {
                    mma_ts(tmem + LY::ACC_A_COL, tmem + (half == 0 ? LY::ds_slice(0, k) : LY::ds_slice(1, k)),
                           y1 + static_cast<uint64_t>((k * 2048) >> 4), IDESC_ACC, k > 0 ? 1u : acc);
                    if (MODE == MODE_DKV)
                        mma_ts(tmem + LY::ACC_B_COL, tmem + (half == 0 ? LY::p_slice(0, k) : LY::p_slice(1, k)),
                               y2 + static_cast<uint64_t>((k * 2048) >> 4), IDESC_ACC, k > 0 ? 1u : acc);
                }
                if (LY::SEP) tc_commit(&bars[LY::BAR_ACC_HALF + half]);
            };
            auto y_full = [&](int g, int code) {         // the copy of half step g has landed
                return wait_warp(LY::BAR_Y_FULL + g % LY::HSTAGES, (g / LY::HSTAGES) & 1, code);
            };
            if (ok) ok = y_full(0, 0x520) && y_full(1, 0x520);
            if (ok) {
                tc_fence_after();
                if (elect_one()) { issue_t(0, 0); issue_t(0, 1); }
                __syncwarp();
            }
            for (int j = 0; j < nsteps && ok; ++j) {
                const bool more = j + 1 < nsteps;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    // (the next half step's copy landed long ago: its barrier is checked before the wait for the
                    // element-wise warps, not behind it, where the check would sit in the chain of the half)
                    if (more) ok = y_full(2 * (j + 1) + half, 0x521);
                    if (ok) ok = wait_warp(LY::BAR_PD_FULL + half, j & 1, 0x530 + half);
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
                        if (LY::SEP && more) issue_t(j + 1, half);
                        issue_acc(j, half);
                        if (!LY::SEP && more) issue_t(j + 1, half);
                        tc_commit(&bars[LY::BAR_Y_EMPTY + (2 * j + half) % LY::HSTAGES]);
                        if (half == 1 && !more) tc_commit(&bars[LY::BAR_ACC_DONE]);
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        // ------------------------------------------------------------ element-wise + epilogue (warps 0-15)
        const int q = warp & 3, h = (warp >> 2) & 1, half = warp >> 3, part = warp >> 2;
        const int r = q * 32 + lane;                     // lane of the TMEM = row of the stationary tile
        const int xr = x0 + r;                           // that row's index (query in MODE_DQ, key in MODE_DKV)
        const uint32_t tl = tmem + (static_cast<uint32_t>(q * 32) << 16);
        const float c2 = scale * LOG2E;
        bool ok = true;
        // Per-lane terms (MODE_DQ): lse of the row in base-2 units (+inf switches a row off: no key, or
        // past the end) and delta = sum_t dO O, each of the row's four warps summing a quarter of the features.
        float lse2_r = INFINITY, delta_r = 0.f;
        if (MODE == MODE_DQ) {
            float sum = 0.f;
            if (xr < Nq) {
                const uint4* a = reinterpret_cast<const uint4*>(dOg + (static_cast<int64_t>(bh) * Nq + xr) * D + part * (D / 4));
                const uint4* b = reinterpret_cast<const uint4*>(Og + (static_cast<int64_t>(bh) * Nq + xr) * D + part * (D / 4));
#pragma unroll
                for (int v = 0; v < D / 32; ++v) {
                    const uint4 av = a[v], bv = b[v];
                    const uint32_t aw[4] = {av.x, av.y, av.z, av.w}, bw[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        sum = fmaf(__uint_as_float(aw[e] << 16), __uint_as_float(bw[e] << 16), sum);
                        sum = fmaf(__uint_as_float(aw[e] & 0xffff0000u), __uint_as_float(bw[e] & 0xffff0000u), sum);
                    }
                }
                const float l = lse[static_cast<int64_t>(bh) * Nq + xr];
                lse2_r = l == -INFINITY ? INFINITY : l * LOG2E;
            }
            xch[part * BT + r] = sum;
            ew_sync();
            delta_r = (xch[r] + xch[BT + r]) + (xch[2 * BT + r] + xch[3 * BT + r]);
            if (part == 0 && xr < Nq) delta[static_cast<int64_t>(bh) * Nq + xr] = delta_r;
        }
        // keys the row takes part with (MODE_DQ: per query row; MODE_DKV: the row IS a key)
        const long long rlim = static_cast<long long>(xr) + 1 + coff;
        const int nrow = rlim < nkeys ? (rlim < 0 ? 0 : static_cast<int>(rlim)) : nkeys;
        const bool key_live = xr < nkeys;
        const uint64_t c22 = pack2(c2, c2);
        const int cq = half * HC + h * 32;               // this warp's 32 columns of every step
        const uint32_t ds_addr = tl + (half == 0 ? LY::ds_store(0, 0) : LY::ds_store(1, 0)) + h * (LY::ds_store(0, 1) - LY::ds_store(0, 0));
        const uint32_t p_addr = tl + (half == 0 ? LY::p_store(0, 0) : LY::p_store(1, 0)) + h * (LY::p_store(0, 1) - LY::p_store(0, 0));
        for (int j = 0; j < nsteps && ok; ++j) {
            if (MODE == MODE_DKV) ok = wait_warp(LY::BAR_VEC_FULL + j % LY::VSTAGES, static_cast<uint32_t>(j / LY::VSTAGES) & 1u, 0x548);
            if (ok) ok = wait_warp(LY::BAR_T_FULL + half, j & 1, 0x540 + half);
            if (!ok) break;
            tc_fence_after();
            const int y0 = (y_begin + j) * BT + cq;      // index of the first of the columns (key or query)
            // all 32 x 32 (row, column) pairs of this warp visible?  (then no per-element selection)
            const bool fast = __all_sync(0xffffffffu, MODE == MODE_DQ ? y0 + 32 <= nrow
                                                                      : key_live && static_cast<long long>(y0) + coff >= xr);
            const float* lv = vec + (j % LY::VSTAGES) * 2 * BT + cq;
            uint32_t pk[16], dk[16];
            // two loads of 16 columns each from T1 and T2 (few registers live at a time)
#pragma unroll
            for (int sub = 0; sub < 2; ++sub) {
                uint32_t t1[16], t2[16];
                tmem_ld_x16(tl + LY::T1_COL + cq + sub * 16, t1);
                tmem_ld_x16(tl + LY::T2_COL + cq + sub * 16, t2);
                tc_wait_ld();
                // p = 2^(c T1 - lse2), ds = p (T2 - delta), on packed pairs (two results per issue slot)
                if (fast) {
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        uint64_t nl[2], dl[2];           // -lse2 and delta of columns i..i+1, i+2..i+3
                        if (MODE == MODE_DQ) {
                            nl[0] = nl[1] = pack2(-lse2_r, -lse2_r);
                            dl[0] = dl[1] = pack2(delta_r, delta_r);
                        } else {
                            const float4 a4 = *reinterpret_cast<const float4*>(lv + sub * 16 + i);
                            const float4 b4 = *reinterpret_cast<const float4*>(lv + BT + sub * 16 + i);
                            nl[0] = pack2(-a4.x, -a4.y); nl[1] = pack2(-a4.z, -a4.w);
                            dl[0] = pack2(b4.x, b4.y); dl[1] = pack2(b4.z, b4.w);
                        }
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int x = i + 2 * e;
                            float a0, a1;
                            unpack2(fma2(pack2(__uint_as_float(t1[x]), __uint_as_float(t1[x + 1])), c22, nl[e]), a0, a1);
                            const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
                            float d0, d1;
                            unpack2(mul2(pack2(p0, p1), sub2(pack2(__uint_as_float(t2[x]), __uint_as_float(t2[x + 1])), dl[e])), d0, d1);
                            if (MODE == MODE_DKV) pk[sub * 8 + x / 2] = pack_bf16x2(p0, p1);
                            dk[sub * 8 + x / 2] = pack_bf16x2(d0, d1);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float p[2], ds[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int col = y0 + sub * 16 + i + e;
                            const float lse2 = MODE == MODE_DQ ? lse2_r : lv[sub * 16 + i + e];
                            const float dl = MODE == MODE_DQ ? delta_r : lv[BT + sub * 16 + i + e];
                            const bool live = MODE == MODE_DQ ? col < nrow : key_live && static_cast<long long>(col) + coff >= xr;
                            p[e] = live ? ex2_approx(fmaf(__uint_as_float(t1[i + e]), c2, -lse2)) : 0.f;
                            ds[e] = p[e] * (__uint_as_float(t2[i + e]) - dl);
                        }
                        pk[sub * 8 + i / 2] = pack_bf16x2(p[0], p[1]);
                        dk[sub * 8 + i / 2] = pack_bf16x2(ds[0], ds[1]);
                    }
                }
            }
            // (own columns for the bf16 tiles: the MMAs that read the previous step's must be done)
            if (LY::SEP && j > 0) {
                ok = wait_warp(LY::BAR_ACC_HALF + half, static_cast<uint32_t>(j - 1) & 1u, 0x542 + half);
                if (!ok) break;
            }
            if (MODE == MODE_DKV) tmem_st_x16(p_addr, pk);
            tmem_st_x16(ds_addr, dk);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[LY::BAR_PD_FULL + half]);
        }
        if (ok && nsteps > 0) ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::BAR_ACC_DONE], 0, abort_flag, status, 0x550));
        if (ok) {
            tc_fence_after();
            // this thread's quarter of the features of its row: acc_a -> outA (dQ, or dK), acc_b -> outB (dV)
#pragma unroll
            for (int o = 0; o < (MODE == MODE_DKV ? 2 : 1); ++o) {
                __nv_bfloat16* out = o == 0 ? outA : outB;
                const float f = o == 0 ? scale : 1.f;
                const uint32_t col = (o == 0 ? LY::ACC_A_COL : LY::ACC_B_COL) + part * (D / 4);
                __nv_bfloat16* orow = out + (static_cast<int64_t>(bh) * NX + xr) * D + part * (D / 4);
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    uint32_t a[16];
                    if (nsteps > 0) {
                        tmem_ld_x16(tl + col + c * 16, a);
                        tc_wait_ld();
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) a[i] = 0u;  // nothing sees this tile: zero gradient
                    }
                    if (xr < NX) {
#pragma unroll
                        for (int v = 0; v < 2; ++v) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(a[8 * v + 0]) * f, __uint_as_float(a[8 * v + 1]) * f);
                            w.y = pack_bf16x2(__uint_as_float(a[8 * v + 2]) * f, __uint_as_float(a[8 * v + 3]) * f);
                            w.z = pack_bf16x2(__uint_as_float(a[8 * v + 4]) * f, __uint_as_float(a[8 * v + 5]) * f);
                            w.w = pack_bf16x2(__uint_as_float(a[8 * v + 6]) * f, __uint_as_float(a[8 * v + 7]) * f);
                            *reinterpret_cast<uint4*>(orow + c * 16 + v * 8) = w;
                        }
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
int launch_bwd_d(const BwdProblem& p, cudaStream_t st) {
    // every tensor is stationary (boxes of 128 rows) in one launch and streamed (boxes of 64 rows) in the other
    CUtensorMap tmQ, tmK, tmV, tmdO, tmQh, tmKh, tmVh, tmdOh;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, D, BT) || !make_map(&tmK, p.K, BH, p.Nk, D, BT) ||
        !make_map(&tmV, p.V, BH, p.Nk, D, BT) || !make_map(&tmdO, p.dO, BH, p.Nq, D, BT) ||
        !make_map(&tmQh, p.Q, BH, p.Nq, D, HC) || !make_map(&tmKh, p.K, BH, p.Nk, D, HC) ||
        !make_map(&tmVh, p.V, BH, p.Nk, D, HC) || !make_map(&tmdOh, p.dO, BH, p.Nq, D, HC))
        return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<bwd_tc_kernel<D, MODE_DQ>>(BL<D, MODE_DQ>::SMEM_BYTES)) return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<bwd_tc_kernel<D, MODE_DKV>>(BL<D, MODE_DKV>::SMEM_BYTES)) return FLAT_ERR_CUDA;
    const int coff = p.causal ? p.Nk - p.Nq : (1 << 30);
    const __nv_bfloat16* dO = static_cast<const __nv_bfloat16*>(p.dO);
    const __nv_bfloat16* O = static_cast<const __nv_bfloat16*>(p.O);
    {
        dim3 grid((p.Nq + BT - 1) / BT, BH);
        bwd_tc_kernel<D, MODE_DQ><<<grid, BWD_THREADS, BL<D, MODE_DQ>::SMEM_BYTES, st>>>(
            tmQ, tmdO, tmKh, tmVh, dO, O, p.lse, p.delta, static_cast<__nv_bfloat16*>(p.dQ), nullptr, p.H, p.Nq, p.Nk,
            p.scale, p.k_valid_len, coff, p.status);
        if (cudaGetLastError() != cudaSuccess) return FLAT_ERR_CUDA;
    }
    {
        dim3 grid((p.Nk + BT - 1) / BT, BH);
        bwd_tc_kernel<D, MODE_DKV><<<grid, BWD_THREADS, BL<D, MODE_DKV>::SMEM_BYTES, st>>>(
            tmK, tmV, tmQh, tmdOh, dO, O, p.lse, p.delta, static_cast<__nv_bfloat16*>(p.dK),
            static_cast<__nv_bfloat16*>(p.dV), p.H, p.Nq, p.Nk, p.scale, p.k_valid_len, coff, p.status);
        if (cudaGetLastError() != cudaSuccess) return FLAT_ERR_CUDA;
    }
    return FLAT_OK;
}

}  // namespace

int launch_bwd_tc(const BwdProblem& p, cudaStream_t st) {
    if (p.d == 64) return launch_bwd_d<64>(p, st);
    if (p.d == 128) return launch_bwd_d<128>(p, st);
    return FLAT_ERR_UNSUPPORTED;
}

}  // namespace flat

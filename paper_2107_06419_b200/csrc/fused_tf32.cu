// Fused Logit-Softmax-Attend for fp32 tensors on the tensor cores (fp32 in, fp32 out, d = 64).
//
// The tensor cores take 32-bit operands only as tf32 (10 mantissa bits), so every fp32 operand x is
// split into x_hi (x with its low 13 mantissa bits cleared: exactly a tf32 number) and
// x_lo = x - x_hi (exact in fp32), and each contraction is the sum of three tf32 products
//     a b  ~=  a_lo b_hi + a_hi b_lo + a_hi b_hi          (the dropped a_lo b_lo is 2^-22 of the result)
// accumulated in fp32.  Both contractions of the path are done this way: S = Q K^T and, per key step,
// P V with the weights P split the same way.  The accumulation ACROSS key steps is not left to the
// tensor core: each step's P V lands in a fresh TMEM buffer and the row's owner thread adds it to the
// running output in registers, O = alpha O + P V, in round-to-nearest fp32 -- the rescaling of the
// streaming softmax then costs nothing extra, and the result does not depend on how the tensor core
// rounds a 16K-term running sum.
//
// Paper mapping (Section 5, 5.1, 5.2): shared outer loops = (batch, head) on blockIdx.y and a tile of
// 128 query rows on blockIdx.x (R-granularity); Logit and Attend run interleaved over 64-key steps with
// the streaming softmax between them; the logits and weights never leave TMEM.
//
// CTA = 512 threads, four warpgroups:
//   warps 0-3  softmax of the even key steps (thread r <-> row r <-> TMEM lane r): Q -> TMEM once (scaled,
//              split), then per step the row maximum, p = 2^(x - m), the split of p into TMEM, and
//              O = alpha O + (P V of its step before)
//   warps 4-7  softmax of the odd key steps, the same way with a running maximum, sum and output of its own:
//              the two streams never talk until the end, where they are merged like two partial softmaxes
//   warps 8-11 converters: warps 8, 9 K tile -> (K_hi in place, K_lo); warps 10, 11 V tile -> transposed
//              (V^T_hi, V^T_lo), since a tf32 operand must have the contraction index contiguous in shared memory
//   warp  12   TMA producer (one lane): Q once, K and raw V tiles into rings
//   warps 13, 14  MMA issuers of the even / odd key steps (one elected lane each): 24 + 24 tcgen05.mma of
//              128 x 64 x 8 per step, A always from TMEM
//   warp  15   idle (it completes the warpgroup for the register hand-over)
// TMEM columns: Q_hi 0, Q_lo 64, S/P_hi 128 + 64 b, P_lo 256 + 64 b, PV 384 + 64 b (b = step parity).
// Every wait is bounded (see tc_common.cuh); on expiry the CTA aborts cleanly and reports a code.
#include <cuda.h>
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
constexpr int BN = 64;               // keys per step
constexpr int D = 64;
constexpr int KS = 3;                // K ring (each stage: K_hi and K_lo tiles)
constexpr int VR = 2;                // raw V ring
constexpr int VS = 3;                // transposed V ring (each stage: V^T_hi and V^T_lo tiles)
constexpr int TILE = BN * D * 4;     // 16 KB: two panels of 64 rows x 128 bytes
constexpr int PANEL = 64 * 128;
constexpr int THREADS = 512;
constexpr int MERGE_STRIDE = 68;      // floats per row of the merge scratch (64 outputs, m, l, padding: 16-byte rows, no bank conflicts)
constexpr uint32_t HI_MASK = 0xffffe000u;

constexpr uint32_t QH_COL = 0, QL_COL = 64, S_COL = 128, PL_COL = 256, PV_COL = 384, TMEM_COLS = 512;

// shared memory: K_hi[KS] K_lo[KS] Vraw[VR] VT_hi[VS] VT_lo[VS]; the Q tile is staged over VT_hi[0..1]
constexpr int OFF_KH = 0, OFF_KL = OFF_KH + KS * TILE, OFF_VR = OFF_KL + KS * TILE, OFF_VTH = OFF_VR + VR * TILE,
              OFF_VTL = OFF_VTH + VS * TILE, TILE_BYTES = OFF_VTL + VS * TILE;
static_assert(VS * TILE >= BM * D * 4, "the Q tile is staged over the V^T_hi ring");
static_assert(2 * KS * TILE >= BM * MERGE_STRIDE * 4, "the merge scratch lies over the K rings");
constexpr int SMEM_BYTES = TILE_BYTES + 512 + 1024;

// barriers
constexpr int Q_FULL = 0, Q_READY = 1, K_FULL = 2, KC_FULL = K_FULL + KS, K_EMPTY = KC_FULL + KS, V_FULL = K_EMPTY + KS,
              VR_EMPTY = V_FULL + VR, VT_FULL = VR_EMPTY + VR, VT_EMPTY = VT_FULL + VS, S_FULL = VT_EMPTY + VS,
              P_FULL = S_FULL + 2, PV_FULL = P_FULL + 2, PV_FREE = PV_FULL + 2, NUM_BARS = PV_FREE + 2;

// D[tmem] (+)= A[tmem] * B[smem desc], tf32 operands
__device__ __forceinline__ void mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Instruction descriptor for kind::tf32, fp32 accumulator, both operands with the contraction index contiguous.
constexpr uint32_t IDESC = (1u << 4) | (2u << 7) | (2u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) |
                           (static_cast<uint32_t>(BM >> 4) << 24);

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t lo_of(uint32_t x) {      // x - x_hi, exact
    return __float_as_uint(__uint_as_float(x) - __uint_as_float(x & HI_MASK));
}

__global__ void __launch_bounds__(THREADS, 1)
fused_tf32_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, float* __restrict__ O, int H, int Nq, int Nk,
                  float scale_log2e, const int32_t* __restrict__ valid_len, int coff, int32_t* status,
                  float* __restrict__ lse) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + TILE_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const uint32_t sb = smem_u32(base);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bh = blockIdx.y;
    const int row0 = blockIdx.x * BM;
    int n = Nk;
    if (valid_len) { n = valid_len[bh / H]; n = n < 0 ? 0 : (n > Nk ? Nk : n); }
    {
        // Causal mask (coff = Nk - Nq; 2^30 = none): row r sees keys j < r + 1 + coff, so the CTA's
        // last row bounds the keys of all its rows.
        const long long lim = static_cast<long long>(row0) + BM + coff;
        if (lim < n) n = lim < 0 ? 0 : static_cast<int>(lim);
    }
    const int ntiles = (n + BN - 1) / BN;

    if (threadIdx.x == 384) {
        for (int i = 0; i < NUM_BARS; ++i) {
            if (i == Q_READY) { mbar_init(&bars[i], 8); continue; }
            const bool by_warps = (i >= KC_FULL && i < K_EMPTY) || (i >= VR_EMPTY && i < VT_EMPTY) ||
                                  (i >= P_FULL && i < PV_FULL) || i >= PV_FREE;
            const bool by_two = (i >= KC_FULL && i < K_EMPTY) || (i >= VR_EMPTY && i < VT_EMPTY);   // (converter warp pairs)
            mbar_init(&bars[i], by_two ? 2 : by_warps ? 4 : 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp >= 12) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
        if (warp == 12) {
            // ------------------------------------------------------------ TMA producer
            if (lane == 0 && ntiles > 0) {
                prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
                bool ok = true;
                int k_issued = 0, v_issued = 0;
                auto load_k = [&](int j) {
                    const int s = j % KS;
                    ok = bounded_wait(&bars[K_EMPTY + s], ((j / KS) & 1) ^ 1, abort_flag, status, 0x600 + s);
                    if (!ok) return;
                    mbar_arrive_expect_tx(&bars[K_FULL + s], TILE);
                    tma_load_3d(base + OFF_KH + s * TILE, &tmK, &bars[K_FULL + s], 0, j * BN, bh);
                    tma_load_3d(base + OFF_KH + s * TILE + PANEL, &tmK, &bars[K_FULL + s], 32, j * BN, bh);
                    k_issued = j + 1;
                };
                auto load_v = [&](int j) {
                    const int s = j % VR;
                    ok = bounded_wait(&bars[VR_EMPTY + s], ((j / VR) & 1) ^ 1, abort_flag, status, 0x610 + s);
                    if (!ok) return;
                    mbar_arrive_expect_tx(&bars[V_FULL + s], TILE);
                    tma_load_3d(base + OFF_VR + s * TILE, &tmV, &bars[V_FULL + s], 0, j * BN, bh);
                    tma_load_3d(base + OFF_VR + s * TILE + PANEL, &tmV, &bars[V_FULL + s], 32, j * BN, bh);
                    v_issued = j + 1;
                };
                mbar_arrive_expect_tx(&bars[Q_FULL], BM * D * 4);
                tma_load_3d(base + OFF_VTH, &tmQ, &bars[Q_FULL], 0, row0, bh);
                tma_load_3d(base + OFF_VTH + BM * 128, &tmQ, &bars[Q_FULL], 32, row0, bh);
                load_k(0);
                if (ntiles > 1) load_k(1);
                for (int j = 0; j < ntiles && ok; ++j) {
                    load_v(j);                               // (never behind a K stage that waits for an older S)
                    if (ok && j + 2 < ntiles) load_k(j + 2);
                }
                if (!ok) {
                    drain_wait(&bars[Q_FULL], 0);
                    for (int j = k_issued > KS ? k_issued - KS : 0; j < k_issued; ++j) drain_wait(&bars[K_FULL + j % KS], (j / KS) & 1);
                    for (int j = v_issued > VR ? v_issued - VR : 0; j < v_issued; ++j) drain_wait(&bars[V_FULL + j % VR], (j / VR) & 1);
                }
            }
        } else if (warp <= 14) {
            // ------------------------------------------------------------ MMA issuers: warp 13 the even key steps, warp 14 the odd
            // ones (the whole warp runs the loop, one lane issues).  Within a parity the order P V(j), S(j+2) is program
            // order; the two parities share nothing but the tensor pipe, and one issues while the other waits.
            const int g = warp - 13;
            if (ntiles > g) {
                const uint64_t kh_desc = make_smem_desc_sw128(sb + OFF_KH, 16, 1024);
                const uint64_t kl_desc = make_smem_desc_sw128(sb + OFF_KL, 16, 1024);
                const uint64_t vh_desc = make_smem_desc_sw128(sb + OFF_VTH, 16, 1024);
                const uint64_t vl_desc = make_smem_desc_sw128(sb + OFF_VTL, 16, 1024);
                bool ok = true;
                auto wait = [&](int bar, uint32_t parity, int code) {
                    if (ok) ok = __all_sync(0xffffffffu, bounded_wait(&bars[bar], parity, abort_flag, status, code));
                    if (ok) tc_fence_after();
                };
                // one 128 x 64 x 64 product: eight k-slices of eight (32 bytes of a 128-byte row each)
                auto product = [&](uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, bool first) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mma_tf32_ts(d_tmem, a_tmem + k * 8, b_desc + static_cast<uint64_t>(((k >> 2) * PANEL + (k & 3) * 32) >> 4),
                                    IDESC, !(first && k == 0));
                };
                auto issue_s = [&](int j) {                  // S(j) = Q K_j^T, small terms first; then release the K stage
                    const int ks = j % KS, b = j & 1;
                    if (elect_one()) {
                        const uint64_t st = static_cast<uint64_t>((ks * TILE) >> 4);
                        product(tmem + S_COL + 64 * b, tmem + QL_COL, kh_desc + st, true);
                        product(tmem + S_COL + 64 * b, tmem + QH_COL, kl_desc + st, false);
                        product(tmem + S_COL + 64 * b, tmem + QH_COL, kh_desc + st, false);
                        tc_commit(&bars[S_FULL + b]);
                        tc_commit(&bars[K_EMPTY + ks]);
                    }
                    __syncwarp();
                };
                auto issue_pv = [&](int j) {                 // PV(j) = P_j V_j into its own buffer; then release the V^T stage
                    const int vs = j % VS, b = j & 1;
                    if (elect_one()) {
                        const uint64_t st = static_cast<uint64_t>((vs * TILE) >> 4);
                        product(tmem + PV_COL + 64 * b, tmem + PL_COL + 64 * b, vh_desc + st, true);
                        product(tmem + PV_COL + 64 * b, tmem + S_COL + 64 * b, vl_desc + st, false);
                        product(tmem + PV_COL + 64 * b, tmem + S_COL + 64 * b, vh_desc + st, false);
                        tc_commit(&bars[PV_FULL + b]);
                        tc_commit(&bars[VT_EMPTY + vs]);
                    }
                    __syncwarp();
                };
                wait(Q_READY, 0, 0x620);
                wait(KC_FULL + g, 0, 0x621);
                if (ok) issue_s(g);
                for (int j = g; j < ntiles && ok; j += 2) {
                    wait(VT_FULL + j % VS, (j / VS) & 1, 0x630);
                    wait(PV_FREE + (j & 1), ((j >> 1) & 1) ^ 1, 0x631);
                    // (the converted keys of step j + 2 are checked here, ahead of the wait for the weights, so that
                    // the check does not sit between the two batches of products)
                    if (j + 2 < ntiles) wait(KC_FULL + (j + 2) % KS, ((j + 2) / KS) & 1, 0x633);
                    wait(P_FULL + (j & 1), (j >> 1) & 1, 0x632);
                    if (ok) issue_pv(j);
                    // (S(j+2) overwrites P_hi(j): it goes behind the products that read it)
                    if (j + 2 < ntiles && ok) issue_s(j + 2);
                }
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ converters (warps 8-11)
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        bool ok = true;
        if (warp < 10) {
            // warps 8, 9: K tile -> K_hi (in place) and K_lo, element by element
            const int ct = threadIdx.x - 256;
            for (int j = 0; j < ntiles && ok; ++j) {
                const int s = j % KS;
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[K_FULL + s], (j / KS) & 1, abort_flag, status, 0x641));
                if (!ok) break;
                const uint32_t kh = sb + OFF_KH + s * TILE, kl = sb + OFF_KL + s * TILE;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const uint32_t off = (ct + 64 * i) * 16;
                    const uint4 v = lds128(kh + off);
                    sts128(kl + off, make_uint4(lo_of(v.x), lo_of(v.y), lo_of(v.z), lo_of(v.w)));
                    sts128(kh + off, make_uint4(v.x & HI_MASK, v.y & HI_MASK, v.z & HI_MASK, v.w & HI_MASK));
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[KC_FULL + s]);
            }
        } else {
            // warps 10, 11: V tile -> transposed V^T_hi, V^T_lo.  4 x 4 blocks: a thread's blocks sit on an XOR
            // diagonal of (key block, feature block), which keeps both the 16-byte reads and the transposed
            // 16-byte writes free of bank conflicts under the 128-byte swizzle.
            const int DB = warp - 10, u = lane & 7, tq = lane >> 3;
            if (ntiles > 0)
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[Q_READY], 0, abort_flag, status, 0x640));   // (Q has left the V^T ring)
            for (int j = 0; j < ntiles && ok; ++j) {
                const int r = j % VR, s = j % VS;
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[V_FULL + r], (j / VR) & 1, abort_flag, status, 0x642));
                if (ok) ok = __all_sync(0xffffffffu, bounded_wait(&bars[VT_EMPTY + s], ((j / VS) & 1) ^ 1, abort_flag, status, 0x643));
                if (!ok) break;
                const uint32_t vr = sb + OFF_VR + r * TILE + DB * PANEL;
#pragma unroll
                for (int KB = 0; KB < 2; ++KB) {
                    const uint32_t vth = sb + OFF_VTH + s * TILE + KB * PANEL, vtl = sb + OFF_VTL + s * TILE + KB * PANEL;
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int dbc = u ^ (tq + 4 * i);         // feature block (chunk) within the panel; key block = u
                        uint32_t in[4][4];
#pragma unroll
                        for (int rr = 0; rr < 4; ++rr) {
                            const int krow = 32 * KB + 4 * u + rr;
                            const uint4 v = lds128(vr + krow * 128 + ((dbc ^ (krow & 7)) << 4));
                            in[rr][0] = v.x; in[rr][1] = v.y; in[rr][2] = v.z; in[rr][3] = v.w;
                        }
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int drow = 32 * DB + 4 * dbc + c;
                            const uint32_t off = drow * 128 + ((u ^ (drow & 7)) << 4);
                            sts128(vth + off, make_uint4(in[0][c] & HI_MASK, in[1][c] & HI_MASK, in[2][c] & HI_MASK, in[3][c] & HI_MASK));
                            sts128(vtl + off, make_uint4(lo_of(in[0][c]), lo_of(in[1][c]), lo_of(in[2][c]), lo_of(in[3][c])));
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&bars[VT_FULL + s]); mbar_arrive(&bars[VR_EMPTY + r]); }
            }
        }
    } else {
        // ------------------------------------------------------------ softmax + output (warps 0-7)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 192;");
        const int g = warp >> 2;                             // 0: even key steps, 1: odd key steps (= TMEM buffer)
        const int r = (warp & 3) * 32 + lane;                // row of the tile <-> TMEM lane
        const int row = row0 + r;
        const uint32_t tl = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        bool ok = true;
        float o[D];
#pragma unroll
        for (int i = 0; i < D; ++i) o[i] = 0.f;
        float m = -INFINITY, l = 0.f, alpha_prev = 0.f;
        const long long rlim = static_cast<long long>(row) + 1 + coff;
        const int nrow = rlim < n ? (rlim < 0 ? 0 : static_cast<int>(rlim)) : n;
        const int nrow_min = __shfl_sync(0xffffffffu, nrow, 0);
        if (ntiles > 0) {
            // Q row -> TMEM, scaled by scale * log2(e) and split: the logits arrive in base-2 units
            // (each softmax group moves one 32-feature panel of the tile)
            ok = __all_sync(0xffffffffu, bounded_wait(&bars[Q_FULL], 0, abort_flag, status, 0x650));
            if (ok) {
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const uint4 v = lds128(sb + OFF_VTH + g * (BM * 128) + r * 128 + ((ch ^ (r & 7)) << 4));
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t x = __float_as_uint(__uint_as_float(w[e]) * scale_log2e);
                        hi[ch * 4 + e] = x & HI_MASK;
                        lo[ch * 4 + e] = lo_of(x);
                    }
                }
                tmem_st_x32(tl + QH_COL + g * 32, hi);
                tmem_st_x32(tl + QL_COL + g * 32, lo);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[Q_READY]);
            }
        }
        auto accumulate = [&](int k) {                       // O = alpha_k O + PV(k)  (k: a step of this group)
            ok = __all_sync(0xffffffffu, bounded_wait(&bars[PV_FULL + g], (k >> 1) & 1, abort_flag, status, 0x660 + g));
            if (!ok) return;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t pv[32];
                tmem_ld_x32(tl + PV_COL + 64 * g + c * 32, pv);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[c * 32 + i] = fmaf(o[c * 32 + i], alpha_prev, __uint_as_float(pv[i]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[PV_FREE + g]);
        };
        for (int j = g; j < ntiles && ok; j += 2) {
            // (the output of this group's previous step first: its products completed before S(j)'s did, and
            // P V(j) cannot be issued before that buffer is free again)
            if (j >= 2) accumulate(j - 2);
            if (!ok) break;
            ok = __all_sync(0xffffffffu, bounded_wait(&bars[S_FULL + g], (j >> 1) & 1, abort_flag, status, 0x670 + g));
            if (!ok) break;
            tc_fence_after();
            uint32_t s[64];
            tmem_ld_x32(tl + S_COL + 64 * g, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
            tmem_ld_x32(tl + S_COL + 64 * g + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
            tc_wait_ld();
            const int col0 = j * BN;
            const int nvalid = nrow > col0 ? (nrow - col0 < BN ? nrow - col0 : BN) : 0;   // per row
            if (col0 + BN > nrow_min) {                      // (warp-uniform) some row has masked keys in this step
#pragma unroll
                for (int i = 0; i < 64; ++i) if (i >= nvalid) s[i] = __float_as_uint(-INFINITY);
            }
            float e0 = __uint_as_float(s[0]), e1 = __uint_as_float(s[1]), e2 = __uint_as_float(s[2]), e3 = __uint_as_float(s[3]);
#pragma unroll
            for (int i = 4; i < 60; i += 8) {
                e0 = max3(e0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
                e1 = max3(e1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
                e2 = max3(e2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
                e3 = max3(e3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
            }
            e0 = max3(e0, __uint_as_float(s[60]), __uint_as_float(s[61]));
            e1 = max3(e1, __uint_as_float(s[62]), __uint_as_float(s[63]));
            const float m_new = fmaxf(m, fmaxf(fmaxf(e0, e1), fmaxf(e2, e3)));
            // (a row that has seen no valid key yet has no maximum: 0 stands in, its weights are 2^-inf = 0)
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            const float alpha = ex2_approx(m - m_use);       // 0 on the row's first valid step
            m = m_new;
            const uint64_t neg_m2 = pack2(-m_use, -m_use);
            uint64_t lsum0 = 0ull, lsum1 = 0ull;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t hi[16], lo[16];
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    float x0, x1;
                    unpack2(add2(pack2(__uint_as_float(s[c * 16 + i]), __uint_as_float(s[c * 16 + i + 1])), neg_m2), x0, x1);
                    hi[i] = __float_as_uint(ex2_approx(x0));
                    hi[i + 1] = __float_as_uint(ex2_approx(x1));
                }
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    lsum0 = add2(lsum0, pack2(__uint_as_float(hi[i]), __uint_as_float(hi[i + 1])));
                    lsum1 = add2(lsum1, pack2(__uint_as_float(hi[i + 2]), __uint_as_float(hi[i + 3])));
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const uint32_t p = hi[i];
                    hi[i] = p & HI_MASK;
                    lo[i] = __float_as_uint(__uint_as_float(p) - __uint_as_float(hi[i]));
                }
                tmem_st_x16(tl + S_COL + 64 * g + c * 16, hi);      // P_hi over the logits
                tmem_st_x16(tl + PL_COL + 64 * g + c * 16, lo);
            }
            float l0, l1, l2, l3;
            unpack2(lsum0, l0, l1);
            unpack2(lsum1, l2, l3);
            l = fmaf(l, alpha, (l0 + l1) + (l2 + l3));
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[P_FULL + g]);
            alpha_prev = alpha;
        }
        {
            // this group's last step
            const int last = ntiles - 1 - ((ntiles - 1 - g) & 1);   // largest j < ntiles with j % 2 == g (negative: none)
            if (ok && last >= 0) accumulate(last);
            // (a single key step leaves the odd group without work: it still waits for that step's products,
            // which read the K ring, before it touches the scratch below)
            if (ok && last < 0 && ntiles > 0)
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[PV_FULL + 0], 0, abort_flag, status, 0x680));
        }
        // Merge of the two streams (both have passed their last P V, so every product that read the K rings
        // has completed and no copy into them is in flight: the scratch lies over them).
        float* scratch = reinterpret_cast<float*>(base + OFF_KH) + r * MERGE_STRIDE;
        if (g == 1) {
#pragma unroll
            for (int v = 0; v < D / 4; ++v)
                *reinterpret_cast<float4*>(scratch + 4 * v) = make_float4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
            scratch[D] = m;
            scratch[D + 1] = ok ? l : __int_as_float(0x7fc00000);
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (g == 0) {
            const float m1 = scratch[D], l1 = scratch[D + 1];
            if (ok && l1 == l1 && row < Nq) {                // (a group that gave up leaves NaN: no output then)
                const float mt = fmaxf(m, m1);
                const float mu = mt == -INFINITY ? 0.f : mt;
                const float a0 = ex2_approx(m - mu), a1 = ex2_approx(m1 - mu);
                const float lt = l * a0 + l1 * a1;
                const float inv = lt > 0.f ? 1.f / lt : 0.f;
                if (lse) lse[static_cast<int64_t>(bh) * Nq + row] = lt > 0.f ? (mt + log2f(lt)) * 0.6931471805599453f : -INFINITY;
                const float w0 = a0 * inv, w1 = a1 * inv;
                float4* orow = reinterpret_cast<float4*>(O + (static_cast<int64_t>(bh) * Nq + row) * D);
#pragma unroll
                for (int v = 0; v < D / 4; ++v) {
                    const float4 q = *reinterpret_cast<const float4*>(scratch + 4 * v);
                    orow[v] = make_float4(o[4 * v] * w0 + q.x * w1, o[4 * v + 1] * w0 + q.y * w1, o[4 * v + 2] * w0 + q.z * w1,
                                          o[4 * v + 3] * w0 + q.w * w1);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// fp32 tensor [BH, N, 64] viewed as 3-D {64, N, BH}; box = 32 floats x rows x 1 (one 128-byte-swizzled panel).
bool make_map_f32(CUtensorMap* m, const void* ptr, int BH, int N, int box_rows) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(BH)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 4, static_cast<cuuint64_t>(N) * D * 4};
    cuuint32_t box[3] = {32, static_cast<cuuint32_t>(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tf32_applies(const Problem& p) {
    return p.dtype == FLAT_DTYPE_F32 && p.d == 64 && !p.bias && !p.block_mask;
}

int launch_fused_tf32(const Problem& p, cudaStream_t st) {
    if (!tf32_applies(p)) return FLAT_ERR_UNSUPPORTED;
    CUtensorMap tmQ, tmK, tmV;
    const int BH = p.B * p.H;
    if (BH > 65535) return FLAT_ERR_SHAPE;      // (grid y)
    if (!make_map_f32(&tmQ, p.Q, BH, p.Nq, BM) || !make_map_f32(&tmK, p.K, BH, p.Nk, BN) ||
        !make_map_f32(&tmV, p.V, BH, p.Nk, BN))
        return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<fused_tf32_kernel>(SMEM_BYTES)) return FLAT_ERR_CUDA;
    dim3 grid((p.Nq + BM - 1) / BM, BH);
    fused_tf32_kernel<<<grid, THREADS, SMEM_BYTES, st>>>(tmQ, tmK, tmV, static_cast<float*>(p.O), p.H, p.Nq, p.Nk,
                                                         p.scale * 1.4426950408889634f, p.k_valid_len,
                                                         p.causal ? p.Nk - p.Nq : (1 << 30), p.status, p.lse);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

}  // namespace flat

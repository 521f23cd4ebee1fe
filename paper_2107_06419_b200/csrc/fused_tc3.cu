// Fused Logit-Softmax-Attend for d = 64 with the softmax of each query tile split over two warps
// per row group and the logit tiles computed three tile-steps ahead (bf16 in, fp32 accumulate,
// bf16 out).  Two query tiles of 128 rows per CTA, as in fused_tc2.cu, but
//   * sixteen softmax warps instead of eight: a thread owns HALF a row of a 128-key step (64
//     logits, exponentiated in place), so every scheduler of the SM holds four softmax warps whose
//     waits (barrier, TMEM load, store completion) hide behind the exponentials of the others;
//   * TMEM holds O_A, O_B (64 columns each) and THREE logit buffers X0..X2 of 128 columns that the
//     tile-steps g = 0, 1, 2, ... of the CTA (g even: tile A, g odd: tile B, key step g / 2, counted
//     over all its work items) use in rotation; the weights P(g) overlay the logits S(g) they came
//     from, and S(g + 3) is issued as soon as the MMAs that read P(g) have completed: the logits
//     of a tile's next step are computed while the other tile's softmax runs.
//
// Paper mapping (Section 5, 5.1, 5.2): shared outer loops = work items (batch, head, slab of 256
// query rows: R-granularity), walked by min(items, SMs) persistent CTAs -- CTA c takes items c,
// c + gridDim.x, ... and its rings, buffers and barrier phases run on across item boundaries;
// inner loops Logit and Attend interleaved over 128-key tiles, the streaming softmax between them.
//
// CTA = 640 threads, five warpgroups; registers move from the fifth to the first four:
//   warps 0-15  softmax: warp w serves row group q = w % 4 (TMEM lanes 32q..32q+31) of tile
//               t = w / 8, key half h = (w / 4) % 2 of every step
//   warp  16    TMA producer (one lane): per item the Q tiles, then K and V tiles into separate rings
//   warp  17/18 MMA issuers (one elected lane each) of O_t += P(g) V for the tile-steps of tile A / B
//   warp  19    MMA issuer of the logits S(g) of both tiles
// The two warps that share a row keep the same reference maximum m_ref: the first step of the CTA's
// first item (and of an item whose first step is partly masked) fixes it from the exact maximum of
// both halves (exchanged through shared memory); every other step reuses the reference it has -- the
// first step of a later item the one carried over from the item before -- and the two warps vote,
// with one reducing named barrier per step, on whether either half's row sum overflowed 2^40 (or,
// on a carried reference, vanished), in which case both redo the step with a fresh common maximum
// (the logits are still in TMEM: the vote comes before the weights are stored over them) and O_t, l
// are rescaled.
// A second instantiation (VL) runs packed batches of sequences of different lengths: the tensor maps
// then view [tokens, H, d] tensors, an item is (sequence, head, slab) and reads its sequence's
// offsets from device arrays (see get_item).
// Every wait is bounded (see tc_common.cuh); on expiry the CTA aborts cleanly and reports a code.
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

constexpr int BM = 128;              // rows per query tile (two tiles per CTA)
constexpr int BN = 128;              // keys per step
constexpr int HN = 64;               // keys per step and softmax thread
constexpr float OVERFLOW_SUM = 1.0995116e12f;   // 2^40: a row sum beyond this means m_ref is stale
constexpr float UNDERFLOW_SUM = 8.6736174e-19f; // 2^-60: a first-step sum below this means a carried m_ref is far too high
// Registers per thread after the hand-over: 640 threads start with 96 each; 512 * 104 + 128 * 64 uses them all.
constexpr int SOFT_REGS = 104, OTHER_REGS = 64;
static_assert(512 * SOFT_REGS + 128 * OTHER_REGS <= 640 * 96, "register hand-over exceeds the CTA's allocation");
constexpr bool USE_POLY = true;          // part of the exponentials on the FMA pipe (see exp_pack_x2)
// bit i: pair i of the 16 pairs (32 logits) of a half step takes the polynomial; two pairs = one element in eight.
// Which pairs is a matter of the instruction schedule only: all 120 two-pair masks were timed on c2 with the
// descending sum loop of exp_pack_x2 (960-986 TFLOP/s), then the 20 mixed choices among the best five.
constexpr unsigned POLY_PAIRS_A = 0x0900, POLY_PAIRS_B = 0x0900;   // first / second 32 logits of a thread's 64
constexpr unsigned PRODUCER_SLEEP = 400; // ns between the TMA producer's probes of a full ring (it runs far ahead: its reaction time is immaterial)

constexpr int D = 64;                // head size of this kernel

struct L3 {
    static constexpr int KS = 4;                         // K ring depth (S runs 1.5 key steps ahead of P V)
    static constexpr int VS = 3;                         // V ring depth
    static constexpr int SOFT_WARPS = 16;
    static constexpr int THREADS = 32 * SOFT_WARPS + 128;
    static constexpr uint32_t TMEM_COLS = 512;
    static constexpr int Q_BYTES = BM * D * 2;           // one query tile
    static constexpr int KV_BYTES = BN * D * 2;
    static constexpr int TILE_BYTES = 2 * Q_BYTES + (KS + VS) * KV_BYTES;
    static constexpr int XCH_BYTES = 2 * 2 * 2 * BM * 4; // [maximum | row sum][tile][half][row] floats
    static constexpr int SMEM_BYTES = TILE_BYTES + XCH_BYTES + 512 + 1024;
    __host__ __device__ static constexpr uint32_t O_COL(int t) { return 64u * t; }
    __host__ __device__ static constexpr uint32_t X_COL(int b) { return 128u + 128u * b; }   // logit / weight buffer b
    // barrier indices
    static constexpr int Q_FULL = 0;                     // [2]
    static constexpr int K_FULL = 2, K_EMPTY = K_FULL + KS;
    static constexpr int V_FULL = K_EMPTY + KS, V_EMPTY = V_FULL + VS;
    // S_FULL / P_FULL / PV_DONE [tile][buffer]: S(u) is in the buffer / P(u) is in the buffer (the 8
    // softmax warps of the tile arrive) / the MMAs that read P(u) have completed.  Tile u & 1 uses
    // buffer u % 3 every sixth tile-step, in phase u / 6.  A buffer's next use starts only behind its
    // PV_DONE, and a tile's softmax warps can be at most two key steps apart, so a waiter never finds
    // one of these barriers more than one phase ahead of the phase it asks for (parity waits are safe).
    static constexpr int S_FULL = V_EMPTY + VS, P_FULL = S_FULL + 6, PV_DONE = P_FULL + 6;
    static constexpr int Q_EMPTY = PV_DONE + 6;          // [2] the item's logit MMAs are done with the Q tile
    static constexpr int NUM_BARS = Q_EMPTY + 2;
};

__device__ __forceinline__ float half_max(const uint32_t (&s)[HN]) {
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
    return fmaxf(fmaxf(e0, e1), fmaxf(e2, e3));
}
__device__ __forceinline__ float half_min(const uint32_t (&s)[HN]) {
    float e0 = __uint_as_float(s[0]), e1 = __uint_as_float(s[1]), e2 = __uint_as_float(s[2]), e3 = __uint_as_float(s[3]);
#pragma unroll
    for (int i = 4; i < 60; i += 8) {
        e0 = min3(e0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        e1 = min3(e1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        e2 = min3(e2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        e3 = min3(e3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
    }
    e0 = min3(e0, __uint_as_float(s[60]), __uint_as_float(s[61]));
    e1 = min3(e1, __uint_as_float(s[62]), __uint_as_float(s[63]));
    return fminf(fminf(e0, e1), fminf(e2, e3));
}

__device__ __forceinline__ void st_shared_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cta.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ float ld_shared_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cta.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}

// Named barrier of the two warps (64 threads) that share a row group of a tile.
__device__ __forceinline__ void pair_sync(int id) {
    asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory");
}
// The same barrier, returning the OR of `flag` over its 64 threads.
__device__ __forceinline__ bool pair_any(int id, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %2, 0;\n\t"
        "bar.red.or.pred p, %1, 64, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(static_cast<uint32_t>(flag))
        : "memory");
    return r != 0;
}

// ex2_poly (see tc_common.cuh) without the upper clamp: the caller keeps the maximum of the
// arguments and treats one above 126 as an overflow of the row.  Scalar on purpose: the constants
// ride along as immediates, where packed instructions would want them in registers.
__device__ __forceinline__ float ex2_poly_lo(float x) {
    x = fmaxf(x, -126.f);
    const float t = x + 12582912.f;                    // 1.5 * 2^23: the low mantissa bits now hold round(x)
    const float f = x - (t - 12582912.f);
    float p = fmaf(0.05508868f, f, 0.24260405f);
    p = fmaf(p, f, 0.69327624f);
    p = fmaf(p, f, 0.99992894f);
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}

// The common case (all 32 logits of a chunk valid) in two parts, so that the registers of the
// logits are free for the next TMEM load while the exponentials run.
// Part 1: x = r * scale + neg_m as packed pairs.
__device__ __forceinline__ void scale32(const uint32_t (&r)[32], uint64_t scale2, uint64_t neg_m2, uint64_t (&x2)[16]) {
#pragma unroll
    for (int i = 0; i < 16; ++i)
        x2[i] = fma2(pack2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), scale2, neg_m2);
}
// Part 2: p = 2^x, packed row sums, bf16 packing.  With POLY, pairs 1, 5, 9, 13 (one element in
// four) take the polynomial instead of the ex2 unit and `xmax` follows the largest argument given
// to it.  l2[0] sums elements 0, 1 (mod 4), l2[1] elements 2, 3.
template <bool POLY, unsigned POLY_PAIRS = POLY_PAIRS_A>
__device__ __forceinline__ void exp_pack_x2(const uint64_t (&x2)[16], uint64_t (&l2)[2], float& xmax, uint32_t (&pk)[16]) {
    float p[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float a, b;
        unpack2(x2[i], a, b);
        if (POLY && ((POLY_PAIRS >> i) & 1)) {
            xmax = max3(xmax, a, b);
            p[2 * i] = ex2_poly_lo(a);
            p[2 * i + 1] = ex2_poly_lo(b);
        } else {
            p[2 * i] = ex2_approx(a);
            p[2 * i + 1] = ex2_approx(b);
        }
    }
    // Descending: the last exponentials issued are summed and packed first. Same sums up to rounding order; the
    // schedule the compiler makes of it is 0.4 % faster on c2 than the ascending loop.
#pragma unroll
    for (int i = 28; i >= 0; i -= 4) {
        l2[0] = add2(l2[0], pack2(p[i], p[i + 1]));
        l2[1] = add2(l2[1], pack2(p[i + 2], p[i + 3]));
        pk[i / 2] = pack_bf16x2(p[i], p[i + 1]);
        pk[i / 2 + 1] = pack_bf16x2(p[i + 2], p[i + 3]);
    }
}

// p_i = 2^(r_i * scale + neg_m) for 32 logits of a row: adds the unrounded p to the four partial
// sums l[] and packs bf16(p) into pk[].  TAIL: only the first `nvalid` logits take part, the rest
// get p = 0 (this also removes the NaN of inf * 0 when scale == 0).  All FFMAs come first, then all
// exponentials, then the sums and the packing, so that consecutive ex2 never wait on a neighbour.
template <bool TAIL, bool POLY>
__device__ __forceinline__ void exp_pack32(const uint32_t (&r)[32], float scale_log2e, float neg_m, int nvalid,
                                           float (&l)[4], uint32_t (&pk)[16]) {
    float p[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) p[i] = fmaf(__uint_as_float(r[i]), scale_log2e, neg_m);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        // One element in four takes the polynomial route (FMA pipe) to unload the ex2 unit.
        p[i] = (!TAIL && POLY && (i & 3) == 3) ? ex2_poly(p[i]) : ex2_approx(p[i]);
        if (TAIL && i >= nvalid) p[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        l[0] += p[i]; l[1] += p[i + 1]; l[2] += p[i + 2]; l[3] += p[i + 3];
        pk[i / 2] = pack_bf16x2(p[i], p[i + 1]);
        pk[i / 2 + 1] = pack_bf16x2(p[i + 2], p[i + 3]);
    }
}

// One work item = (batch, head, slab of 256 query rows).  A CTA takes the items blockIdx.x,
// blockIdx.x + gridDim.x, ... one after the other without draining its pipeline in between.
struct Item {
    int bh, row0, n, ntiles;                             // n = number of keys that any row of the slab sees, ntiles = key steps
    bool skip;                                           // an empty slot of the paired order: no rows to write either
    // packed variable-length batches only:
    int head, q_tok0, k_tok0, q_rows, coff;              // head; first token of the slab's rows / of the sequence's keys; rows of the sequence from row0 on; Nk - Nq of the sequence
};
// What every role needs to enumerate the items.
struct Sched {
    int items, slabs, H, Nk;
    const int32_t* valid_len;
    int coff;                                            // causal mask: row r sees keys j < r + 1 + coff (coff = Nk - Nq); none: 2^30
    int paired;                                          // items come in pairs of complementary slabs (see get_item)
    const int32_t* cu_q;                                 // packed variable-length batches: first token of every sequence's
    const int32_t* cu_k;                                 // queries / keys in the packed tensors ([sequences + 1] entries)
};
// The sequence of item indices of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...; in paired mode the
// CTA takes PAIRS of consecutive indices (2 c, 2 c + 1), (2 (c + gridDim.x), ...), ...
__device__ __forceinline__ int first_item(const Sched& sc) { return sc.paired ? 2 * blockIdx.x : blockIdx.x; }
__device__ __forceinline__ int next_item(int idx, const Sched& sc) {
    return sc.paired ? ((idx & 1) ? idx - 1 + 2 * static_cast<int>(gridDim.x) : idx + 1) : idx + static_cast<int>(gridDim.x);
}
// VL (packed variable-length batches): Q, O are [total_q, H, d], K, V [total_k, H, d]; sequence s owns
// tokens cu_q[s] .. cu_q[s+1] - 1 of Q and cu_k[s] .. cu_k[s+1] - 1 of K, V.  Item index =
// (sequence * H + head) * slabs + slab with `slabs` taken from the longest sequence; a slab past the
// end of its sequence is an empty slot.  The causal offset is that of the sequence.
template <bool VL>
__device__ __forceinline__ Item get_item(int idx, const Sched& sc) {
    Item it;
    int slab;
    bool empty = false;
    if (VL) {
        it.bh = idx / sc.slabs;
        slab = idx - it.bh * sc.slabs;
        const int s = it.bh / sc.H;
        it.head = it.bh - s * sc.H;
        const int q0 = sc.cu_q[s], ql = sc.cu_q[s + 1] - q0, k0 = sc.cu_k[s], kl = sc.cu_k[s + 1] - k0;
        it.row0 = slab * (2 * BM);
        it.q_tok0 = q0 + it.row0;
        it.k_tok0 = k0;
        it.q_rows = ql - it.row0;
        it.coff = sc.coff < (1 << 29) ? kl - ql : sc.coff;
        it.skip = it.q_rows <= 0;
        int n = kl < 0 ? 0 : kl;
        const long long lim = static_cast<long long>(it.row0) + 2 * BM + it.coff;
        n = lim < n ? (lim < 0 ? 0 : static_cast<int>(lim)) : n;
        if (it.skip) n = 0;
        it.n = n;
        it.ntiles = (n + BN - 1) / BN;
        return it;
    }
    if (sc.paired) {
        // Under the causal mask a slab's work grows with its position.  A persistent CTA walks a fixed
        // share of the items, so the shares must weigh the same: the slabs of a head are taken in
        // pairs (p, slabs - 1 - p), whose key counts add up to the same total for every p, and a CTA
        // always takes both members.  Index = head * slots + 2 p + member; with an odd number of
        // slabs the middle one is its own partner and its second slot stays empty.
        const int slots = (sc.slabs + 1) & ~1;
        it.bh = idx / slots;
        const int i = idx - it.bh * slots, p = i >> 1;
        slab = (i & 1) ? sc.slabs - 1 - p : p;
        empty = (i & 1) && slab == p;
    } else {
        it.bh = idx / sc.slabs;
        slab = idx - it.bh * sc.slabs;
        // (one CTA per item under the causal mask: rotate the order of the slabs from head to head, so
        // that CTAs launched together do not all hold slabs of the same length)
        if (sc.coff < (1 << 29)) slab = (slab + 7 * it.bh) % sc.slabs;
    }
    it.row0 = slab * (2 * BM);
    int n = sc.Nk;
    if (sc.valid_len) { n = sc.valid_len[it.bh / sc.H]; n = n < 0 ? 0 : (n > sc.Nk ? sc.Nk : n); }
    // under the causal mask the slab's last row bounds the keys of the item
    const long long lim = static_cast<long long>(it.row0) + 2 * BM + sc.coff;
    n = lim < n ? (lim < 0 ? 0 : static_cast<int>(lim)) : n;
    if (empty) n = 0;
    it.skip = empty;
    it.n = n;
    it.ntiles = (n + BN - 1) / BN;
    return it;
}
// Position of a role in the CTA's sequence of key steps.  Items without a valid key have no steps
// and are skipped (their rows are written as zeros by the softmax warps).  J counts the key steps
// of all items so far: the rings, the buffers and the barrier phases are indexed with it, so the
// pipeline runs on across item boundaries; q counts the items that had steps (phase of the Q tiles).
struct Cursor {
    int idx, j, J, q;
    Item it;
    bool valid;
};
template <bool VL>
__device__ __forceinline__ void cursor_seek(Cursor& c, const Sched& sc) {
    c.valid = false;
    while (c.idx < sc.items) {
        c.it = get_item<VL>(c.idx, sc);
        if (c.it.ntiles > 0) { c.valid = true; return; }
        c.idx = next_item(c.idx, sc);
    }
}
template <bool VL>
__device__ __forceinline__ void cursor_init(Cursor& c, const Sched& sc) {
    c.idx = first_item(sc); c.j = 0; c.J = 0; c.q = 0;
    cursor_seek<VL>(c, sc);
}
template <bool VL>
__device__ __forceinline__ void cursor_next(Cursor& c, const Sched& sc) {
    ++c.j; ++c.J;
    if (c.j == c.it.ntiles) {
        c.j = 0; ++c.q;
        c.idx = next_item(c.idx, sc);
        cursor_seek<VL>(c, sc);
    }
}

// VL: packed variable-length batches (see get_item); the tensor maps then view the packed tensors as
// {d, H, tokens} and valid_len is unused (cu_k gives the key counts).
// WLSE: also writes lse[b,h,i] = log of row i's sum of exponentials (dense batches; what the
// backward pass takes from the forward one).  A separate instantiation, so that the plain forward
// kernel is compiled exactly as it is without the output.
template <bool VL, bool WLSE = false>
__global__ void __launch_bounds__(L3::THREADS, 1)
fused_tc3_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, int H, int Nq, int Nk,
                 int items, int slabs, float scale_log2e, const int32_t* __restrict__ valid_len, int coff,
                 int32_t* status, int wide_stores, int paired, const int32_t* __restrict__ cu_q,
                 const int32_t* __restrict__ cu_k, float* __restrict__ lse) {
    using LY = L3;
    const Sched sc{items, slabs, H, Nk, valid_len, coff, paired, cu_q, cu_k};
    if (VL && static_cast<int>(gridDim.x) == items) {
        // one CTA per slot: a slot past the end of its sequence leaves before anything is set up
        if (get_item<VL>(blockIdx.x, sc).skip) return;
    }
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Qs = base;                                  // 2 tiles
    uint8_t* Ks = Qs + 2 * LY::Q_BYTES;                  // KS tiles
    uint8_t* Vs = Ks + LY::KS * LY::KV_BYTES;            // VS tiles
    float* xch = reinterpret_cast<float*>(base + LY::TILE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + LY::TILE_BYTES + LY::XCH_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + LY::NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == LY::SOFT_WARPS * 32) {
        for (int i = 0; i < LY::NUM_BARS; ++i)
            mbar_init(&bars[i], (i >= LY::P_FULL && i < LY::PV_DONE) ? 8               // one arrival per softmax warp of the tile
                                : (i >= LY::V_EMPTY && i < LY::S_FULL) ? 2 : 1);   // V_EMPTY: both O += P V issuers
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, LY::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp >= LY::SOFT_WARPS) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(OTHER_REGS));
      const uint32_t bars_s = smem_u32(bars), abort_s = smem_u32(const_cast<int*>(abort_flag));
      if (warp == LY::SOFT_WARPS) {
        // ------------------------------------------------------------ TMA producer
        // Per item: Q_A, K_0, Q_B, K_1, then V_j and K_{j+2} in turn (S runs ahead of P V, so K_{j+2} is
        // wanted before V_{j+1}).  The rings are indexed with the global key step J.
        if (lane == 0) {
            prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
            bool ok = true;
            int q_loaded[2] = {0, 0}, k_issued = 0, v_issued = 0;    // (for the drain after a failed wait)
            // (y, z): coordinates of the tile in the tensor map beyond the feature index -- (row, head of
            // the batch), or (head, token) for packed batches
            auto load_q = [&](int t, int q, int y, int z) {
                // the logit MMAs of the previous item must have finished with this tile of shared memory
                if (q > 0) ok = bounded_wait_s<PRODUCER_SLEEP>(bars_s + 8 * (LY::Q_EMPTY + t), (q - 1) & 1, abort_s, status, 0x120 + t);
                if (!ok) return;
                mbar_arrive_expect_tx(&bars[LY::Q_FULL + t], LY::Q_BYTES);
                tma_load_3d(Qs + t * LY::Q_BYTES, &tmQ, &bars[LY::Q_FULL + t], 0, y, z);
                q_loaded[t] = q + 1;
            };
            auto load_k = [&](int J, int y, int z) {
                const int s = J % LY::KS;
                ok = bounded_wait_s<PRODUCER_SLEEP>(bars_s + 8 * (LY::K_EMPTY + s), ((J / LY::KS) & 1) ^ 1, abort_s, status, 0x100 + s);
                if (!ok) return;
                mbar_arrive_expect_tx(&bars[LY::K_FULL + s], LY::KV_BYTES);
                tma_load_3d(Ks + s * LY::KV_BYTES, &tmK, &bars[LY::K_FULL + s], 0, y, z);
                k_issued = J + 1;
            };
            auto load_v = [&](int J, int y, int z) {
                const int s = J % LY::VS;
                ok = bounded_wait_s<PRODUCER_SLEEP>(bars_s + 8 * (LY::V_EMPTY + s), ((J / LY::VS) & 1) ^ 1, abort_s, status, 0x110 + s);
                if (!ok) return;
                mbar_arrive_expect_tx(&bars[LY::V_FULL + s], LY::KV_BYTES);
                tma_load_3d(Vs + s * LY::KV_BYTES, &tmV, &bars[LY::V_FULL + s], 0, y, z);
                v_issued = J + 1;
            };
            int J0 = 0, q = 0;
            for (int idx = first_item(sc); idx < items && ok; idx = next_item(idx, sc)) {
                const Item it = get_item<VL>(idx, sc);
                if (it.ntiles == 0) continue;
                // tile of query rows r.. / of keys of step j
                auto qy = [&](int r) { return VL ? it.head : r; };
                auto qz = [&](int r) { return VL ? it.q_tok0 + (r - it.row0) : it.bh; };
                auto ky = [&](int j) { return VL ? it.head : j * BN; };
                auto kz = [&](int j) { return VL ? it.k_tok0 + j * BN : it.bh; };
                load_q(0, q, qy(it.row0), qz(it.row0));
                if (ok) load_k(J0, ky(0), kz(0));
                if (ok) load_q(1, q, qy(it.row0 + BM), qz(it.row0 + BM));
                if (ok && it.ntiles > 1) load_k(J0 + 1, ky(1), kz(1));
                for (int j = 0; j < it.ntiles && ok; ++j) {
                    load_v(J0 + j, ky(j), kz(j));
                    if (ok && j + 2 < it.ntiles) load_k(J0 + j + 2, ky(j + 2), kz(j + 2));
                }
                J0 += it.ntiles;
                ++q;
            }
            if (!ok) {
                for (int t = 0; t < 2; ++t)
                    if (q_loaded[t] > 0) drain_wait(&bars[LY::Q_FULL + t], (q_loaded[t] - 1) & 1);
                for (int J = k_issued > LY::KS ? k_issued - LY::KS : 0; J < k_issued; ++J)
                    drain_wait(&bars[LY::K_FULL + J % LY::KS], (J / LY::KS) & 1);
                for (int J = v_issued > LY::VS ? v_issued - LY::VS : 0; J < v_issued; ++J)
                    drain_wait(&bars[LY::V_FULL + J % LY::VS], (J / LY::VS) & 1);
            }
        }
      } else {
        // ------------------------------------------------------------ MMA issuers
        // Warp 17 / 18 issues O_t += P(g) V for the tile-steps of tile A / B; warp 19 issues every
        // logit tile S(g), into buffer g % 3, once the O += P V of tile-step g - 3 (same buffer, the
        // other tile) has read its weights.  Three warps, so that none of the three streams of MMAs
        // queues behind a wait that belongs to another.  A whole warp runs the loop (uniform
        // control flow); one elected lane issues.  Tile-step g = 2 J + tile
        // (J: global key step), buffer g % 3, barrier phase g / 6.
        constexpr uint32_t IDESC_S = make_idesc_bf16(BM, BN, 0, 0);
        constexpr uint32_t IDESC_PV = make_idesc_bf16(BM, D, 0, 1);
        bool ok = true;
        auto wait = [&](int bar, uint32_t parity, int code) {
            if (ok) ok = __all_sync(0xffffffffu, bounded_wait_s(bars_s + 8 * bar, parity, abort_s, status, code));
            if (ok) tc_fence_after();
        };
        Cursor c;
        cursor_init<VL>(c, sc);
        if (warp == LY::SOFT_WARPS + 3) {
            const uint64_t q_desc = make_smem_desc_sw128(smem_u32(Qs), 16, 1024);
            const uint64_t k_desc = make_smem_desc_sw128(smem_u32(Ks), 16, 1024);
            while (c.valid && ok) {
                const int ks = c.J % LY::KS;
                wait(LY::K_FULL + ks, (c.J / LY::KS) & 1, 0x210);
#pragma unroll
                for (int ts = 0; ts < 2; ++ts) {
                    const int g = 2 * c.J + ts, bs = g % 3;
                    if (c.j == 0) wait(LY::Q_FULL + ts, c.q & 1, 0x200 + ts);
                    // buffer bs was last used by tile-step g - 3, of the other tile
                    if (g >= 3) wait(LY::PV_DONE + (ts ^ 1) * 3 + bs, ((g - 3) / 6) & 1, 0x230 + ts);
                    if (!ok) break;
                    if (elect_one()) {
                        const uint64_t qd = q_desc + static_cast<uint64_t>((ts * LY::Q_BYTES) >> 4);
                        const uint64_t kd = k_desc + static_cast<uint64_t>((ks * LY::KV_BYTES) >> 4);
#pragma unroll
                        for (int k = 0; k < D / 16; ++k)
                            mma_ss(tmem + LY::X_COL(bs), qd + static_cast<uint64_t>((k * 32) >> 4),
                                   kd + static_cast<uint64_t>((k * 32) >> 4), IDESC_S, k > 0);
                        tc_commit(&bars[LY::S_FULL + ts * 3 + bs]);
                        if (ts == 1) tc_commit(&bars[LY::K_EMPTY + ks]);          // both tiles' logits have used K_j
                        if (c.j == c.it.ntiles - 1) tc_commit(&bars[LY::Q_EMPTY + ts]);   // the item's last use of Q_ts
                    }
                    __syncwarp();
                }
                cursor_next<VL>(c, sc);
            }
        } else {
            const int t = warp - LY::SOFT_WARPS - 1;
            const uint64_t v_desc = make_smem_desc_sw128(smem_u32(Vs), BN * 128, 1024);
            while (c.valid && ok) {
                const int g = 2 * c.J + t, b = g % 3, vs = c.J % LY::VS;
                wait(LY::V_FULL + vs, (c.J / LY::VS) & 1, 0x220);
                wait(LY::P_FULL + t * 3 + b, (g / 6) & 1, 0x221);
                if (!ok) break;
                if (elect_one()) {
                    const uint64_t vd = v_desc + static_cast<uint64_t>((vs * LY::KV_BYTES) >> 4);
                    // the two halves of P(g) overlay the first 32 columns of each half of S(g)
#pragma unroll
                    for (int k = 0; k < BN / 16; ++k)
                        mma_ts(tmem + LY::O_COL(t), tmem + LY::X_COL(b) + (k / 4) * HN + (k % 4) * 8,
                               vd + static_cast<uint64_t>((k * 2048) >> 4), IDESC_PV, (c.j > 0 || k > 0));
                    tc_commit(&bars[LY::PV_DONE + t * 3 + b]);
                    tc_commit(&bars[LY::V_EMPTY + vs]);
                }
                __syncwarp();
                cursor_next<VL>(c, sc);
            }
        }
      }
    } else {
        // ------------------------------------------------------------ softmax + epilogue (warps 0-15)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(SOFT_REGS));
        const int q = warp & 3;                          // row group = TMEM lane quarter
        const int t = warp >> 3;                         // query tile
        const int h = (warp >> 2) & 1;                   // key half of every step
        const uint32_t tl = tmem + (static_cast<uint32_t>(q * 32) << 16);
        const int pair_id = 1 + t * 4 + q;               // named barrier of the two warps sharing these rows
        // shared-window addresses: the barriers, the abort flag, and this thread's slot for exchanged
        // maxima (its partner's is BM floats away: flip bit 9; the row sums sit 4 * BM floats further)
        const uint32_t bars_s = smem_u32(bars), abort_s = smem_u32(const_cast<int*>(abort_flag));
        const uint32_t xm_own = smem_u32(xch + ((t * 2 + h) * BM + q * 32 + lane));
        const bool neg_scale = scale_log2e < 0.f;
        bool ok = true;
        int b = t;                                       // buffer of tile-step g = 2 J + t: g % 3
        int g = t;                                       // this tile's next tile-step (J: key steps of all items so far)
        // The reference maximum is carried from item to item: any reference gives the exact softmax
        // as long as the sums neither overflow nor vanish, and the rows of the next item mostly have
        // logits of the same size, so its first step can skip the exact maximum too.  The first item
        // of the CTA and items whose first step is partly masked start from an exact maximum.
        float m_ref = -INFINITY;
        bool first_item_done = false;
        for (int idx = first_item(sc); idx < items; idx = next_item(idx, sc)) {
        const Item it = get_item<VL>(idx, sc);
        if (it.skip) continue;
        const int ntiles = it.ntiles;
        // keys this thread's row sees (all the item's keys unless the causal mask cuts the row short);
        // lane 0 has the shortest row of the warp, so its count tells whether a step needs the masked routine
        const long long rlim = static_cast<long long>(it.row0) + t * BM + q * 32 + lane + 1 + (VL ? it.coff : sc.coff);
        const int nrow = rlim < it.n ? (rlim < 0 ? 0 : static_cast<int>(rlim)) : it.n;
        const int nrow_min = __shfl_sync(0xffffffffu, nrow, 0);
        float l = 0.f;
        const bool exact_first = !first_item_done || sc.coff < (1 << 29) || it.n < BN;   // (the same for all warps)
        first_item_done = true;
        for (int j = 0; j < ntiles; ++j, g += 2, b = (b == 0 ? 2 : b - 1)) {      // g += 2  <=>  b -= 1 (mod 3)
            // this warp's 64 logits of S(g); its 32 packed columns of P(g) go over the first half of them
            const uint32_t s_addr = tl + LY::X_COL(b) + h * HN;
            const uint32_t xph = static_cast<uint32_t>(g / 6) & 1u;   // phase parity of this tile's use of the buffer
            // A warp whose wait fails does not leave by itself: it goes on to the next vote with its
            // partner (reading TMEM that may not be ready is harmless, nothing is stored), so that the
            // two always pass the same sequence of named barriers and leave together.
            ok = bounded_wait_s(bars_s + 8 * (LY::S_FULL + t * 3 + b), xph, abort_s, status, 0x300 + t);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            const int col0 = j * BN + h * HN;
            const bool tail = col0 + HN > nrow_min;      // (warp-uniform) some row has masked keys in this step
            const int nvalid = nrow > col0 ? (nrow - col0 < HN ? nrow - col0 : HN) : 0;   // per row
            // p = 2^(scale*s - m_ref); row sum in fp32 from the unrounded p; P rounded to bf16.  Any
            // reference m_ref gives the exact softmax, so the common case takes no row maximum; a sum
            // beyond 2^40 (or inf/NaN) in either half shows that the reference fell too far behind,
            // and both halves then redo the step the careful way.  The logits stay in TMEM until the
            // two warps have voted, so the redo reads them again instead of holding them in registers.
            uint32_t pk[2][16];
            float ls[4] = {0.f, 0.f, 0.f, 0.f};
            bool careful = (j == 0) && exact_first;
            if (!careful) {
                // (the logits come in two loads of 32 so that few registers are live at a time)
                uint32_t r[32];
                float lt;
                tmem_ld_x32(s_addr, r);
                tc_wait_ld();
                if (tail) {
                    exp_pack32<true, false>(r, scale_log2e, -m_ref, nvalid, ls, pk[0]);
                    tmem_ld_x32(s_addr + 32, r);
                    tc_wait_ld();
                    exp_pack32<true, false>(r, scale_log2e, -m_ref, nvalid - 32, ls, pk[1]);
                    lt = (ls[0] + ls[1]) + (ls[2] + ls[3]);
                } else {
                    const uint64_t scale2 = pack2(scale_log2e, scale_log2e), neg_m2 = pack2(-m_ref, -m_ref);
                    uint64_t l2[2] = {0ull, 0ull};
                    uint64_t x2[16];
                    float xmax = 0.f;
                    scale32(r, scale2, neg_m2, x2);
                    tmem_ld_x32(s_addr + 32, r);         // the second 32 logits arrive during the first 32 exponentials
                    exp_pack_x2<USE_POLY>(x2, l2, xmax, pk[0]);
                    tc_wait_ld();
                    scale32(r, scale2, neg_m2, x2);
                    exp_pack_x2<USE_POLY, POLY_PAIRS_B>(x2, l2, xmax, pk[1]);
                    float a, b2, c, d2;
                    unpack2(l2[0], a, b2);
                    unpack2(l2[1], c, d2);
                    lt = (a + b2) + (c + d2);
                    ls[0] = lt;
                    if (xmax > 126.f) lt = INFINITY;      // the polynomial was fed an argument beyond its range
                }
                // (a first step on a carried reference must also show that the reference is not far
                // ABOVE the row's logits: its sum must not have vanished)
                careful = pair_any(pair_id, !(lt <= OVERFLOW_SUM) || (j == 0 && !(lt >= UNDERFLOW_SUM)) || !ok);
            }
            if (careful) {
                if (pair_any(pair_id, !ok)) { ok = false; break; }     // (both warps are here: j == 0 or the joint vote)
                if (j == 0) m_ref = -INFINITY;           // nothing accumulated yet: the item starts from its own maximum
                float mx = -INFINITY;
                {
                    uint32_t s[HN];
                    tmem_ld_x32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
                    tmem_ld_x32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
                    tc_wait_ld();
                    if (tail) {
                        const uint32_t excl = __float_as_uint(neg_scale ? INFINITY : -INFINITY);
#pragma unroll
                        for (int i = 0; i < HN; ++i) if (i >= nvalid) s[i] = excl;
                    }
                    if (nvalid > 0) mx = (neg_scale ? half_min(s) : half_max(s)) * scale_log2e;
                }
                st_shared_f32(xm_own, mx);
                pair_sync(pair_id);
                mx = fmaxf(mx, ld_shared_f32(xm_own ^ (BM * 4)));
                if (__any_sync(0xffffffffu, mx > m_ref + RESCALE_THRESHOLD)) {
                    const float m_new = fmaxf(m_ref, mx);
                    // 0 on the first step; a row that has not seen a valid key yet (causal mask) keeps l = 0
                    const float alpha = m_new == -INFINITY ? 1.f : ex2_approx(m_ref - m_new);
                    l *= alpha;
                    if (j > 0) {
                        // each half rescales its half of the columns of O_t
                        // (O_t += P(g - 2) V must be complete; that tile-step used buffer b + 1 mod 3)
                        const int u2 = g - 2;
                        ok = __all_sync(0xffffffffu,
                                        bounded_wait_s(bars_s + 8 * (LY::PV_DONE + t * 3 + (b == 2 ? 0 : b + 1)),
                                                       static_cast<uint32_t>(u2 / 6) & 1u, abort_s, status, 0x310 + t));
                        if (ok) {
                            tc_fence_after();
#pragma unroll
                            for (int c = 0; c < D / 64; ++c) {
                                uint32_t r[32];
                                const uint32_t addr = tl + LY::O_COL(t) + h * (D / 2) + c * 32;
                                tmem_ld_x32(addr, r);
                                tc_wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                                tmem_st_x32(addr, r);
                            }
                        }
                    }
                    m_ref = m_new;
                }
                // the logits are read again, 32 at a time; with the fresh maximum every argument is <= 0,
                // so the ordinary routine (polynomial lanes included) applies unless part of the half is masked
                ls[0] = ls[1] = ls[2] = ls[3] = 0.f;
                if (tail) {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(s_addr + c * 32, r);
                        tc_wait_ld();
                        exp_pack32<true, false>(r, scale_log2e, -m_ref, nvalid - c * 32, ls, pk[c]);
                    }
                } else {
                    const uint64_t scale2 = pack2(scale_log2e, scale_log2e), neg_m2 = pack2(-m_ref, -m_ref);
                    uint64_t l2[2] = {0ull, 0ull};
                    float xmax = 0.f;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t r[32];
                        uint64_t x2[16];
                        tmem_ld_x32(s_addr + c * 32, r);
                        tc_wait_ld();
                        scale32(r, scale2, neg_m2, x2);
                        exp_pack_x2<USE_POLY>(x2, l2, xmax, pk[c]);
                    }
                    float a, b2, c2, d2;
                    unpack2(l2[0], a, b2);
                    unpack2(l2[1], c2, d2);
                    ls[0] = (a + b2) + (c2 + d2);
                }
            }
            // a failed wait is voted on so that the two warps leave the loop together (only the
            // careful path waits for anything)
            if (careful && pair_any(pair_id, !ok)) ok = false;
            if (!ok) break;
            tmem_st_x16(s_addr, pk[0]);
            tmem_st_x16(s_addr + 16, pk[1]);
            l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_s(bars_s + 8 * (LY::P_FULL + t * 3 + b));
        }
        if (ok && ntiles > 0) {
            // the last O_t += P V of the item (the issuer's MMAs complete in order)
            const int ul = g - 2;
            ok = bounded_wait_s(bars_s + 8 * (LY::PV_DONE + t * 3 + (b == 2 ? 0 : b + 1)), static_cast<uint32_t>(ul / 6) & 1u,
                                abort_s, status, 0x330 + t);
            ok = __all_sync(0xffffffffu, ok);
        }
        // The two warps of a row leave together if either gave up; otherwise they add up their row sums.
        if (pair_any(pair_id, !ok)) { ok = false; break; }
        st_shared_f32(xm_own + 4 * BM * 4, l);
        pair_sync(pair_id);
        l += ld_shared_f32((xm_own ^ (BM * 4)) + 4 * BM * 4);
        {
            const int row = it.row0 + t * BM + q * 32 + lane;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            // (m_ref, common to the row's two warps, and the exponents are in base-2 units)
            if (WLSE && h == 0 && row < Nq)
                lse[static_cast<int64_t>(it.bh) * Nq + row] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            tc_fence_after();
            // (packed batches: token-major [tokens, H, d])
            __nv_bfloat16* orow = VL ? O + ((static_cast<int64_t>(it.q_tok0) + (row - it.row0)) * H + it.head) * D + h * (D / 2)
                                     : O + (static_cast<int64_t>(it.bh) * Nq + row) * D + h * (D / 2);
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                uint32_t r[32];
                if (ntiles > 0) {
                    tmem_ld_x32(tl + LY::O_COL(t) + h * (D / 2) + c * 32, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;      // no valid key: O = 0
                }
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    w[i] = pack_bf16x2(__uint_as_float(r[2 * i]) * inv, __uint_as_float(r[2 * i + 1]) * inv);
                if (!VL && wide_stores) {                // (O is 32-byte aligned; dense layout: rows 128 bytes apart)
                    // Lane pairs swap one 32-byte sector each, so that a store instruction of the warp covers 16 rows
                    // x 64 contiguous bytes instead of 32 rows x 32 bytes: the load/store unit takes a store one line
                    // at a time, and the sixteen warps' stores are what an item boundary waits for.
                    const bool odd = lane & 1;
                    uint32_t a[8], b[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t got = __shfl_xor_sync(0xffffffffu, odd ? w[i] : w[8 + i], 1);   // odd lanes give their first sector, even lanes their second
                        a[i] = odd ? got : w[i];         // first instruction: the even lane's row (own first sector / the partner's second)
                        b[i] = odd ? w[8 + i] : got;     // second instruction: the odd lane's row
                    }
                    const int row_e = row - (odd ? 1 : 0);
                    __nv_bfloat16* even_row = orow - (odd ? D : 0);
                    if (row_e < Nq) st_global_32B(even_row + c * 32 + (odd ? 16 : 0), a);
                    if (row_e + 1 < Nq) st_global_32B(even_row + D + c * 32 + (odd ? 16 : 0), b);
                } else if (VL ? row - it.row0 < it.q_rows : row < Nq) {
                    if (wide_stores) {
                        st_global_32B(orow + c * 32, *reinterpret_cast<uint32_t(*)[8]>(&w[0]));
                        st_global_32B(orow + c * 32 + 16, *reinterpret_cast<uint32_t(*)[8]>(&w[8]));
                    } else {
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) =
                                make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
                    }
                }
            }
            // (the reads of O_t above are complete -- tcgen05.wait::ld -- before this warp's next P_FULL
            // arrival, which the first, overwriting O_t = P V of the next item waits for)
            tc_fence_before();
        }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, LY::TMEM_COLS);
}

int launch_tc3(const Problem& p, cudaStream_t st) {
    using LY = L3;
    CUtensorMap tmQ, tmK, tmV;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, D, BM) || !make_map(&tmK, p.K, BH, p.Nk, D, BN) ||
        !make_map(&tmV, p.V, BH, p.Nk, D, BN))
        return FLAT_ERR_CUDA;
    if (!(p.lse ? ensure_dynamic_smem<fused_tc3_kernel<false, true>>(LY::SMEM_BYTES)
                : ensure_dynamic_smem<fused_tc3_kernel<false, false>>(LY::SMEM_BYTES)))
        return FLAT_ERR_CUDA;
    // Work items = (head, 256-row slab), slabs of a head next to each other so that CTAs running at
    // the same time share K and V in L2.  With many items per SM the grid is one persistent CTA per
    // SM, each walking over its share (the fixed deal costs little then and the pipeline never
    // drains); with few, one CTA per item, which the hardware hands out as SMs become free -- the
    // better balance when the items differ in length (key-padding masks) and there are only a few
    // rounds of them.
    const int slabs = (p.Nq + 2 * BM - 1) / (2 * BM);
    const int64_t items = static_cast<int64_t>(slabs) * BH;
    const int sms = device_sm_count();
    // (items of equal length: two per CTA are enough for the fixed deal to pay; under a key-padding
    // mask the items differ in length and the hardware's hand-out balances better until there are many)
    const bool persistent = items >= (p.k_valid_len ? 8 : 2) * static_cast<int64_t>(sms);
    // Persistent CTAs under the causal mask take the slabs of a head in complementary pairs, so that
    // every CTA's share weighs the same (get_item); the item index then runs over slots, two per pair.
    const int paired = persistent && p.causal ? 1 : 0;
    const int64_t slots = paired ? static_cast<int64_t>((slabs + 1) & ~1) * BH : items;
    if (slots > 0x7fffffff) return FLAT_ERR_SHAPE;
    const int grid = static_cast<int>(persistent ? sms : items);
    auto kern = p.lse ? fused_tc3_kernel<false, true> : fused_tc3_kernel<false, false>;
    kern<<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk,
                                                    static_cast<int>(slots), slabs, p.scale * 1.4426950408889634f,
                                                    p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status,
                                                    (reinterpret_cast<uintptr_t>(p.O) & 31) == 0 ? 1 : 0, paired, nullptr,
                                                    nullptr, p.lse);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}


}  // namespace

int launch_fused_tc3_varlen(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_q,
                            const int32_t* cu_k, int num_seqs, int H, int64_t total_q, int64_t total_k,
                            int max_seqlen_q, float scale, int causal, int32_t* status, cudaStream_t st) {
    using LY = L3;
    CUtensorMap tmQ, tmK, tmV;
    if (!make_map_packed(&tmQ, Q, total_q, H, D, BM) || !make_map_packed(&tmK, K, total_k, H, D, BN) ||
        !make_map_packed(&tmV, V, total_k, H, D, BN))
        return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<fused_tc3_kernel<true>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
    const int slabs = (max_seqlen_q + 2 * BM - 1) / (2 * BM);
    const int64_t items = static_cast<int64_t>(slabs) * num_seqs * H;
    if (items > 0x7fffffff) return FLAT_ERR_SHAPE;
    const int sms = device_sm_count();
    // Sequences of different lengths make items of different weight, and a persistent CTA's share is
    // fixed: with long sequences (many slabs, many key steps per item) one CTA per item, handed out by
    // the hardware as SMs become free, balances better (measured on a mix of 8 sequences of 3.9K-14.5K
    // tokens: 2.81 against 2.89 ms, causal 1.61 against 1.86 ms); with many short ones the persistent
    // grid saves the per-CTA set-up.
    const bool persistent = items >= 8 * static_cast<int64_t>(sms) && slabs < 8;
    const int grid = static_cast<int>(persistent ? sms : items);
    fused_tc3_kernel<true><<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(
        tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(O), H, max_seqlen_q, 0, static_cast<int>(items), slabs,
        scale * 1.4426950408889634f, nullptr, causal ? 0 : (1 << 30), status,
        (reinterpret_cast<uintptr_t>(O) & 31) == 0 ? 1 : 0, 0, cu_q, cu_k, nullptr);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

int launch_fused_tc3(const Problem& p, cudaStream_t st) {
    if (p.dtype != FLAT_DTYPE_BF16 || p.d != D) return FLAT_ERR_UNSUPPORTED;
    return launch_tc3(p, st);
}

}  // namespace flat

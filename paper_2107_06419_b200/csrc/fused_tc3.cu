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

#include <mutex>

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
constexpr unsigned POLY_PAIRS_SA = 0x0900, POLY_PAIRS_SB = 0x0900; // the same for the even-deal instantiation (timed on c5)
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
    static constexpr int SMEM_BYTES = TILE_BYTES + XCH_BYTES + 512 + 512 + 1024;   // (.. barriers, the even deal's table, alignment)
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
    int tile0;                                           // first key step of the item that this CTA takes (even deal: see EvenDeal)
    // packed variable-length batches only:
    int head, q_tok0, k_tok0, q_rows, coff;              // head; first token of the slab's rows / of the sequence's keys; rows of the sequence from row0 on; Nk - Nq of the sequence
};
// The even deal (template parameter SPLIT), for launches whose items would fill the SMs badly when dealt whole:
// few items of different length (key-padding masks: the hardware hands out whole items, and the last SM to get
// a long one finishes long after the others), or a number of equal items that leaves the last round mostly empty.
// Every item (b, h, slab) has L_b key steps (at least one, so that a batch without valid keys still gets its
// zero rows written); the key steps of all items, T of them in item order, are cut into gridDim.x equal ranges
// and CTA c takes steps c T / grid .. (c + 1) T / grid - 1: the end of one item, whole items, the beginning of
// one more.  The CTA whose range holds an item's first key step writes the item's rows; every other part of the
// item leaves its un-normalised (m_ref, l, O) in the workspace slot of its CTA -- a CTA has at most one such
// part, its first -- and raises that slot's flags to the launch's epoch, and the writer merges them (the
// split-merge identity of the streaming softmax).  A CTA works through its range in order, so the part it leaves
// for somebody else comes first and the part it must wait for others on comes last; CTA c only ever waits for
// CTAs of a higher number: no cycle, and every wait is bounded.
// Teams: the slabs of a head read the same K and V, and CTAs that hold them at the same key step share those
// tiles in L2.  Dealt item by item, neighbouring CTAs would sit at different key steps of the same head and every
// tile would come from DRAM once per slab (measured: no gain at all on the masked workload).  So the unit that is
// dealt is the head -- all its slabs -- and a team of `team` = slabs CTAs takes a range of head key steps, member
// s of the team working on slab s; team = 1 deals single items.
struct EvenDeal {
    int team;
    int epoch;
    float* ws;                                           // [gridDim.x][WS_FLOATS]
    int* flags;                                          // [gridDim.x][16 softmax warps]
};
// A slot of the workspace: O as [tile][key half][row group][32 columns][32 lanes] fp32, then per tile, key half
// and row group 32 reference maxima and 32 row sums -- every thread reads back what the thread of the same role
// wrote, so a warp waits for the flag of the other CTA's warp of the same number and for nothing else.
constexpr int WS_O_FLOATS = 2 * 2 * 4 * 32 * 32, WS_FLOATS = WS_O_FLOATS + 2 * 2 * 4 * 64;
constexpr int WS_MAX_CTAS = 160;
// The deal's table in shared memory (filled by one warp before the roles start): this CTA's range lo, hi, its
// first item and the one after its last, T, and from DEAL_PREFIX on the number of key steps before batch b's
// items for b = 0 .. B (DEAL_MAX_B batches at most).
constexpr int DEAL_LO = 0, DEAL_HI = 1, DEAL_FIRST = 2, DEAL_END = 3, DEAL_T = 4, DEAL_TEAM = 5, DEAL_TEAMS = 6, DEAL_PREFIX = 8, DEAL_MAX_B = 64;
static_assert((DEAL_PREFIX + DEAL_MAX_B + 1) * 4 <= 512, "the deal's table has 512 bytes of shared memory");
// What every role needs to enumerate the items.
struct Sched {
    int items, slabs, H, Nk;
    const int32_t* valid_len;
    int coff;                                            // causal mask: row r sees keys j < r + 1 + coff (coff = Nk - Nq); none: 2^30
    int paired;                                          // items come in pairs of complementary slabs (see get_item)
    const int32_t* cu_q;                                 // packed variable-length batches: first token of every sequence's
    const int32_t* cu_k;                                 // queries / keys in the packed tensors ([sequences + 1] entries)
    const int* deal;                                     // even deal: its table in shared memory
    EvenDeal ed;
};
// Even deal: first key step of team g's range, of `teams` (g T < 2^32: the launcher checks).
__device__ __forceinline__ int deal_lo(int T, int g, int teams) {
    return static_cast<int>(static_cast<unsigned>(g) * static_cast<unsigned>(T) / static_cast<unsigned>(teams));
}
// Even deal: where item idx (its unit: the item, or its head) sits in the sequence of all key steps.
__device__ __forceinline__ void deal_item_range(const Sched& sc, int idx, int& start, int& end) {
    const int team = sc.deal[DEAL_TEAM], u = idx / team;
    const int per = sc.H * sc.slabs / team, b = u / per, k = u - b * per;
    const int p0 = sc.deal[DEAL_PREFIX + b], Lb = (sc.deal[DEAL_PREFIX + b + 1] - p0) / per;
    start = p0 + k * Lb;
    end = start + Lb;
}
// Even deal: what the softmax warps do with the rows of item idx when this CTA's key steps of it are done:
// 0 normalise and store them (the CTA had the whole item), 2 leave them in this CTA's slot, 1 merge the slots of
// CTAs first, first + team, ... (count of them: the same member of the following teams, whose ranges cover the
// rest of the item) and store.
__device__ __forceinline__ void deal_role(const Sched& sc, int idx, int& part, int& first, int& count) {
    int start, end;
    deal_item_range(sc, idx, start, end);
    const int team = sc.deal[DEAL_TEAM], teams = sc.deal[DEAL_TEAMS], g = static_cast<int>(blockIdx.x) / team;
    part = 0; first = static_cast<int>(blockIdx.x) + team; count = 0;
    if (sc.deal[DEAL_LO] > start) { part = 2; return; }
    if (sc.deal[DEAL_HI] < end) {
        const int T = sc.deal[DEAL_T];
        while (g + 1 + count < teams && deal_lo(T, g + 1 + count, teams) < end) ++count;
        part = count > 0 ? 1 : 0;
    }
}
// A warp waits until `*flag` holds the launch's epoch (lane 0 polls; bounded like every other wait of the kernel).
__device__ __forceinline__ bool wait_flag_warp(const int* flag, int epoch, uint32_t abort_addr, int32_t* status, int code) {
    bool ok = true;
    if ((threadIdx.x & 31) == 0) {
        const long long t0 = clock64();
        for (;;) {
            int v, aborted;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
            if (v == epoch) break;
            asm volatile("ld.volatile.shared::cta.s32 %0, [%1];" : "=r"(aborted) : "r"(abort_addr) : "memory");
            if (aborted) { ok = false; break; }
            if (clock64() - t0 > WAIT_CYCLES) {
                asm volatile("st.volatile.shared::cta.s32 [%0], %1;" ::"r"(abort_addr), "r"(1) : "memory");
                if (status) atomicExch(status, code);
                ok = false;
                break;
            }
            __nanosleep(100);
        }
    }
    ok = __all_sync(0xffffffffu, ok);
    __syncwarp();
    __threadfence();
    return ok;
}
// A part that begins inside its item: the un-normalised rows (this thread: 32 columns of one row, from TMEM
// address `o_addr`), their reference and their sums go to this CTA's slot for the CTA that holds the item's
// beginning.  `role` = (tile * 2 + key half) * 4 + row group.
__device__ __forceinline__ void deal_write_partial(const EvenDeal ed, uint32_t o_addr, int role, float m_ref, float l) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* slot = ed.ws + static_cast<size_t>(blockIdx.x) * WS_FLOATS;
    float* po = slot + role * 1024 + lane;
    float* pm = slot + WS_O_FLOATS + role * 64 + lane;
    uint32_t r[32];
    tmem_ld_x32(o_addr, r);
    tc_wait_ld();
#pragma unroll
    for (int i = 0; i < 32; ++i) po[i * 32] = __uint_as_float(r[i]);
    pm[0] = m_ref;
    pm[32] = l;
    __threadfence();
    __syncwarp();
    if (lane == 0)
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(ed.flags + blockIdx.x * 16 + warp), "r"(ed.epoch) : "memory");
}
// The part that begins its item: (m, l, O) of two parts merge as m = max, l = sum of l_i 2^(m_i - m), O likewise
// (the row-wise softmax of Section 5.2, split along the keys); then 1/l and the store of this thread's 32 columns.
// A part without a valid key carries m = -inf and l = 0 and drops out of the merge.
__device__ __forceinline__ void deal_finish_merged(const EvenDeal ed, uint32_t o_addr, int role, float m_ref, float l, int pfirst,
                                                int pcount, __nv_bfloat16* orow, bool row_valid, uint32_t abort_s, int32_t* status) {
    // (partner CTAs: pfirst, pfirst + team, ...)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t r[32];
    tmem_ld_x32(o_addr, r);
    tc_wait_ld();
    float mm = m_ref;
    for (int pi = 0; pi < pcount; ++pi) {
        const int cp = pfirst + pi * ed.team;
        if (!wait_flag_warp(ed.flags + cp * 16 + warp, ed.epoch, abort_s, status, 0x360)) break;
        const float* slot = ed.ws + static_cast<size_t>(cp) * WS_FLOATS;
        const float* po = slot + role * 1024 + lane;
        const float* pm = slot + WS_O_FLOATS + role * 64 + lane;
        const float m2 = __ldcg(pm), l2 = __ldcg(pm + 32);
        const float mn = fmaxf(mm, m2);
        const float fa = mm == -INFINITY ? 0.f : ex2_approx(mm - mn), fb = m2 == -INFINITY ? 0.f : ex2_approx(m2 - mn);
        l = l * fa + l2 * fb;
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * fa + __ldcg(po + i * 32) * fb);
        mm = mn;
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    if (row_valid) {
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                w[i] = pack_bf16x2(__uint_as_float(r[8 * v + 2 * i]) * inv, __uint_as_float(r[8 * v + 2 * i + 1]) * inv);
            *reinterpret_cast<uint4*>(orow + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}
// The sequence of item indices of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...; in paired mode the
// CTA takes PAIRS of consecutive indices (2 c, 2 c + 1), (2 (c + gridDim.x), ...), ...
template <bool SPLIT = false>
__device__ __forceinline__ int first_item(const Sched& sc) {
    if (SPLIT) return sc.deal[DEAL_FIRST];
    return sc.paired ? 2 * blockIdx.x : blockIdx.x;
}
template <bool SPLIT = false>
__device__ __forceinline__ int next_item(int idx, const Sched& sc) {
    if (SPLIT) return idx + sc.deal[DEAL_TEAM];
    return sc.paired ? ((idx & 1) ? idx - 1 + 2 * static_cast<int>(gridDim.x) : idx + 1) : idx + static_cast<int>(gridDim.x);
}
// VL (packed variable-length batches): Q, O are [total_q, H, d], K, V [total_k, H, d]; sequence s owns
// tokens cu_q[s] .. cu_q[s+1] - 1 of Q and cu_k[s] .. cu_k[s+1] - 1 of K, V.  Item index =
// (sequence * H + head) * slabs + slab with `slabs` taken from the longest sequence; a slab past the
// end of its sequence is an empty slot.  The causal offset is that of the sequence.
template <bool VL, bool SPLIT = false>
__device__ __forceinline__ Item get_item(int idx, const Sched& sc) {
    Item it;
    int slab;
    bool empty = false;
    it.tile0 = 0;
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
    if (SPLIT) {
        // this CTA's share of the item's key steps (an item without a valid key counts one step, fully masked)
        int start, end;
        deal_item_range(sc, idx, start, end);
        const int lo = sc.deal[DEAL_LO] > start ? sc.deal[DEAL_LO] : start, hi = sc.deal[DEAL_HI] < end ? sc.deal[DEAL_HI] : end;
        it.tile0 = lo - start;
        it.ntiles = hi - lo;
    }
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
template <bool VL, bool SPLIT = false>
__device__ __forceinline__ void cursor_seek(Cursor& c, const Sched& sc) {
    c.valid = false;
    while (c.idx < sc.items) {
        c.it = get_item<VL, SPLIT>(c.idx, sc);
        if (c.it.ntiles > 0) { c.valid = true; return; }
        c.idx = next_item<SPLIT>(c.idx, sc);
    }
}
template <bool VL, bool SPLIT = false>
__device__ __forceinline__ void cursor_init(Cursor& c, const Sched& sc) {
    c.idx = first_item<SPLIT>(sc); c.j = 0; c.J = 0; c.q = 0;
    cursor_seek<VL, SPLIT>(c, sc);
}
template <bool VL, bool SPLIT = false>
__device__ __forceinline__ void cursor_next(Cursor& c, const Sched& sc) {
    ++c.j; ++c.J;
    if (c.j == c.it.ntiles) {
        c.j = 0; ++c.q;
        c.idx = next_item<SPLIT>(c.idx, sc);
        cursor_seek<VL, SPLIT>(c, sc);
    }
}

// VL: packed variable-length batches (see get_item); the tensor maps then view the packed tensors as
// {d, H, tokens} and valid_len is unused (cu_k gives the key counts).
// WLSE: also writes lse[b,h,i] = log of row i's sum of exponentials (dense batches; what the
// backward pass takes from the forward one).  A separate instantiation, so that the plain forward
// kernel is compiled exactly as it is without the output.
// SPLIT: the even deal by key steps (see EvenDeal; dense batches, no causal mask, B <= DEAL_MAX_B; `items` is the
// number of items, B * H * slabs, and the grid must not exceed the SMs that can hold a CTA each).
template <bool VL, bool WLSE = false, bool SPLIT = false>
__global__ void __launch_bounds__(L3::THREADS, 1)
fused_tc3_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, int H, int Nq, int Nk,
                 int items, int slabs, float scale_log2e, const int32_t* __restrict__ valid_len, int coff,
                 int32_t* status, int wide_stores, int paired, const int32_t* __restrict__ cu_q,
                 const int32_t* __restrict__ cu_k, float* __restrict__ lse, const EvenDeal ed) {
    using LY = L3;
    static_assert(!SPLIT || (!VL && !WLSE), "the even deal is built for the plain dense forward kernel only");
    Sched sc{items, slabs, H, Nk, valid_len, coff, paired, cu_q, cu_k, nullptr, ed};
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
    int* deal = reinterpret_cast<int*>(base + LY::TILE_BYTES + LY::XCH_BYTES + 512);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == LY::SOFT_WARPS * 32) {
        for (int i = 0; i < LY::NUM_BARS; ++i)
            mbar_init(&bars[i], (i >= LY::P_FULL && i < LY::PV_DONE) ? 8               // one arrival per softmax warp of the tile
                                : (i >= LY::V_EMPTY && i < LY::S_FULL) ? 2 : 1);   // V_EMPTY: both O += P V issuers
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, LY::TMEM_COLS); tmem_relinquish(); }
    if (SPLIT && warp == 1) {
        // The deal's table.  Batch b's items have L_b = max(1, key steps of its valid keys) steps each; two
        // batches per lane, prefix sums by shuffles.
        const int team = ed.team, teams = static_cast<int>(gridDim.x) / team;
        const int B = items / (H * slabs), per = H * slabs / team;      // units (items or heads) per batch
        int v[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int b = lane + 32 * k;
            int n = Nk;
            if (valid_len && b < B) { n = valid_len[b]; n = n < 0 ? 0 : (n > Nk ? Nk : n); }
            const int L = (n + BN - 1) / BN;
            v[k] = b < B ? (L > 0 ? L : 1) * per : 0;
        }
        int carry = 0;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            int x = v[k];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, x, o);
                if (lane >= o) x += y;
            }
            deal[DEAL_PREFIX + 1 + lane + 32 * k] = carry + x;          // steps before batch lane + 32 k + 1
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        __syncwarp();
        if (lane == 0) {
            deal[DEAL_PREFIX] = 0;
            const int T = deal[DEAL_PREFIX + B];
            // (CTAs beyond the last whole team have nothing to do)
            const int g = static_cast<int>(blockIdx.x) / team, member = static_cast<int>(blockIdx.x) - g * team;
            const int lo = g < teams ? deal_lo(T, g, teams) : 0, hi = g < teams ? deal_lo(T, g + 1, teams) : 0;
            // the unit that holds key step x: the batch by its prefix, the unit within the batch by division
            auto unit_of = [&](int x) {
                int b = 0;
                while (b + 1 < B && deal[DEAL_PREFIX + b + 1] <= x) ++b;
                const int p0 = deal[DEAL_PREFIX + b], Lb = (deal[DEAL_PREFIX + b + 1] - p0) / per;
                return b * per + (x - p0) / Lb;
            };
            deal[DEAL_LO] = lo; deal[DEAL_HI] = hi; deal[DEAL_T] = T; deal[DEAL_TEAM] = team; deal[DEAL_TEAMS] = teams;
            deal[DEAL_FIRST] = hi > lo ? unit_of(lo) * team + member : 0;
            deal[DEAL_END] = hi > lo ? (unit_of(hi - 1) + 1) * team : 0;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (SPLIT) { sc.deal = deal; sc.items = deal[DEAL_END]; items = deal[DEAL_END]; }

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
            for (int idx = first_item<SPLIT>(sc); idx < items && ok; idx = next_item<SPLIT>(idx, sc)) {
                const Item it = get_item<VL, SPLIT>(idx, sc);
                if (it.ntiles == 0) continue;
                // tile of query rows r.. / of keys of step j
                auto qy = [&](int r) { return VL ? it.head : r; };
                auto qz = [&](int r) { return VL ? it.q_tok0 + (r - it.row0) : it.bh; };
                auto ky = [&](int j) { return VL ? it.head : (it.tile0 + j) * BN; };
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
        cursor_init<VL, SPLIT>(c, sc);
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
                cursor_next<VL, SPLIT>(c, sc);
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
                cursor_next<VL, SPLIT>(c, sc);
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
        for (int idx = first_item<SPLIT>(sc); idx < items; idx = next_item<SPLIT>(idx, sc)) {
        const Item it = get_item<VL, SPLIT>(idx, sc);
        if (it.skip) continue;
        const int ntiles = it.ntiles;
        // keys this thread's row sees (all the item's keys unless the causal mask cuts the row short);
        // lane 0 has the shortest row of the warp, so its count tells whether a step needs the masked routine
        const long long rlim = static_cast<long long>(it.row0) + t * BM + q * 32 + lane + 1 + (VL ? it.coff : sc.coff);
        // (a part of the even deal counts its keys from its own first step)
        const int nrow_item = rlim < it.n ? (rlim < 0 ? 0 : static_cast<int>(rlim)) : it.n;
        const int nrow = SPLIT ? (nrow_item > it.tile0 * BN ? nrow_item - it.tile0 * BN : 0) : nrow_item;
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
                    exp_pack_x2<USE_POLY, SPLIT ? POLY_PAIRS_SA : POLY_PAIRS_A>(x2, l2, xmax, pk[0]);
                    tc_wait_ld();
                    scale32(r, scale2, neg_m2, x2);
                    exp_pack_x2<USE_POLY, SPLIT ? POLY_PAIRS_SB : POLY_PAIRS_B>(x2, l2, xmax, pk[1]);
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
        if (SPLIT) {
            // an item shared with other CTAs (inlined: with these paths as called functions c5 ran 2 % slower,
            // with the deal's index arithmetic out of line as well 6 %)
            int part, pfirst, pcount;
            deal_role(sc, idx, part, pfirst, pcount);
            if (part != 0) {
                tc_fence_after();
                if (part == 2)
                    deal_write_partial(sc.ed, tl + LY::O_COL(t) + h * (D / 2), (t * 2 + h) * 4 + q, m_ref, l);
                else
                    deal_finish_merged(sc.ed, tl + LY::O_COL(t) + h * (D / 2), (t * 2 + h) * 4 + q, m_ref, l, pfirst, pcount,
                                       O + (static_cast<int64_t>(it.bh) * Nq + it.row0 + t * BM + q * 32 + lane) * D + h * (D / 2),
                                       it.row0 + t * BM + q * 32 + lane < Nq, abort_s, status);
                tc_fence_before();
                continue;
            }
        }
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

// The even deal's workspace: one slot and sixteen flags per CTA, in the library's own device memory (nothing is
// allocated at run time).  The flags hold the epoch of the launch that last wrote the slot; epochs only grow, so
// nothing is ever reset.  One workspace per device: a launch may use it when no launch from another stream can
// still be using it (an event recorded behind every user tells), and not during stream capture (a captured launch
// could be replayed beside anything); otherwise the launch deals whole items as before.
__device__ float g_deal_ws[static_cast<size_t>(WS_MAX_CTAS) * WS_FLOATS];
__device__ int g_deal_flags[WS_MAX_CTAS * 16];
struct DealOwner {
    bool ready = false, used = false;
    float* ws = nullptr;
    int* flags = nullptr;
    cudaEvent_t ev = nullptr;
    cudaStream_t last = nullptr;
};
std::mutex g_deal_mu;
DealOwner g_deal[64];
int g_deal_epoch = 0;

// Fills `ed` (workspace, flags, a fresh epoch) if a launch on `st` may use the current device's workspace; the
// caller launches and calls deal_release() while `lock` is still held.
bool deal_acquire(cudaStream_t st, EvenDeal& ed, std::unique_lock<std::mutex>& lock) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
        cudaGetLastError();                              // (e.g. the legacy stream while another stream captures: not our launch's error)
        return false;
    }
    if (cap != cudaStreamCaptureStatusNone) return false;
    lock = std::unique_lock<std::mutex>(g_deal_mu);
    DealOwner& o = g_deal[dev];
    if (!o.ready) {
        void *w = nullptr, *f = nullptr;
        if (cudaGetSymbolAddress(&w, g_deal_ws) != cudaSuccess || cudaGetSymbolAddress(&f, g_deal_flags) != cudaSuccess ||
            cudaEventCreateWithFlags(&o.ev, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            lock.unlock();
            return false;
        }
        o.ws = static_cast<float*>(w);
        o.flags = static_cast<int*>(f);
        o.ready = true;
    }
    if (o.used && o.last != st && cudaEventQuery(o.ev) != cudaSuccess) {
        cudaGetLastError();                              // (not ready: another stream's launch may still be running)
        lock.unlock();
        return false;
    }
    ed.ws = o.ws;
    ed.flags = o.flags;
    if (g_deal_epoch == 0x7fffffff) g_deal_epoch = 0;
    ed.epoch = ++g_deal_epoch;
    return true;
}
void deal_release(cudaStream_t st) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
    DealOwner& o = g_deal[dev];
    o.used = cudaEventRecord(o.ev, st) == cudaSuccess;
    o.last = st;
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
    // Too few items for the fixed deal: whole items handed out by the hardware leave SMs idle when the items differ
    // in length (key-padding masks) or when the last round is mostly empty; the key steps are dealt evenly instead
    // (EvenDeal), if the average share is long enough to carry the two extra item boundaries.
    if (!persistent && !p.causal && !p.lse && p.B <= DEAL_MAX_B && sms <= WS_MAX_CTAS && items > 0) {
        const int64_t nt = (p.Nk + BN - 1) / BN, rounds = (items + sms - 1) / sms;
        const bool ragged = p.k_valid_len != nullptr || 4 * items < 3 * rounds * sms;   // (unmasked: under three quarters of the rounds filled)
        // teams of `slabs` CTAs if they fill nine SMs in ten; single items only where K and V of all heads stay in L2
        EvenDeal ed{};
        const bool teams_fit = slabs <= sms && 10 * ((sms / slabs) * slabs) >= 9 * sms;
        const bool kv_in_l2 = 4 * static_cast<int64_t>(BH) * p.Nk * D <= (48ll << 20);
        ed.team = teams_fit ? slabs : 1;
        std::unique_lock<std::mutex> lock;
        if (ragged && (teams_fit || kv_in_l2) && items * nt >= 16 * static_cast<int64_t>(sms) && items * nt * (sms + 1) < (1ll << 32) &&
            ensure_dynamic_smem<fused_tc3_kernel<false, false, true>>(LY::SMEM_BYTES) && deal_acquire(st, ed, lock)) {
            fused_tc3_kernel<false, false, true><<<sms, LY::THREADS, LY::SMEM_BYTES, st>>>(
                tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, static_cast<int>(items), slabs,
                p.scale * 1.4426950408889634f, p.k_valid_len, 1 << 30, p.status,
                (reinterpret_cast<uintptr_t>(p.O) & 31) == 0 ? 1 : 0, 0, nullptr, nullptr, nullptr, ed);
            const bool launched = cudaGetLastError() == cudaSuccess;
            deal_release(st);
            g_last_schedule = FLAT_SCHEDULE_EVEN_DEAL;
            return launched ? FLAT_OK : FLAT_ERR_CUDA;
        }
    }
    g_last_schedule = persistent ? FLAT_SCHEDULE_PERSISTENT : FLAT_SCHEDULE_ITEMS;
    auto kern = p.lse ? fused_tc3_kernel<false, true> : fused_tc3_kernel<false, false>;
    kern<<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk,
                                                    static_cast<int>(slots), slabs, p.scale * 1.4426950408889634f,
                                                    p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status,
                                                    (reinterpret_cast<uintptr_t>(p.O) & 31) == 0 ? 1 : 0, paired, nullptr,
                                                    nullptr, p.lse, EvenDeal{});
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}


}  // namespace

thread_local int g_last_schedule = 0;

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
    g_last_schedule = persistent ? FLAT_SCHEDULE_PERSISTENT : FLAT_SCHEDULE_ITEMS;
    fused_tc3_kernel<true><<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(
        tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(O), H, max_seqlen_q, 0, static_cast<int>(items), slabs,
        scale * 1.4426950408889634f, nullptr, causal ? 0 : (1 << 30), status,
        (reinterpret_cast<uintptr_t>(O) & 31) == 0 ? 1 : 0, 0, cu_q, cu_k, nullptr, EvenDeal{});
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

int launch_fused_tc3(const Problem& p, cudaStream_t st) {
    if (p.dtype != FLAT_DTYPE_BF16 || p.d != D) return FLAT_ERR_UNSUPPORTED;
    return launch_tc3(p, st);
}

}  // namespace flat

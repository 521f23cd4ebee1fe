// Fused Logit-Softmax-Attend, pipelined (bf16 in, fp32 accumulate, bf16 out): NT = 2 query tiles
// of 128 rows per CTA share the tensor pipe, the K/V stream and the SM's exponent unit (NT = 1: one
// tile per CTA, two CTAs per SM, for problems too small to fill the SMs with 256-row CTAs).
//
// Paper mapping (Section 5, 5.1, 5.2): shared outer loops = (batch, head) on blockIdx.y and a
// slab of NT x 128 query rows on blockIdx.x (R-granularity); inner loops Logit and Attend run
// interleaved over 128-key tiles with the streaming softmax between them (a reference maximum and
// a running sum replace the paper's full-row on-chip slice; same function).
//
// CTA (NT = 2) = 384 threads, three warpgroups; registers are moved from the third to the first two:
//   warps 0-3  softmax of query tile A   (thread r <-> row r of the tile <-> TMEM lane r)
//   warps 4-7  softmax of query tile B
//   warp  8    TMA producer (one lane): Q tiles once, then K and V tiles into separate rings
//   warp  9    MMA issuer of tile A (one elected lane): S_A = Q_A K^T and O_A += P_A V
//   warp  10   MMA issuer of tile B
//   warp  11   idle (it only completes the warpgroup for the register hand-over)
// A softmax thread pulls its 128 logits into registers and releases the S buffer at once (so the
// next S_t is computed while it works), computes p = 2^(scale*log2e*s - m_ref) with the reference
// maximum it already has -- no row maximum per tile: a tile whose row sum overflows 2^40 is redone
// with an exact maximum, and O_t, l are rescaled -- writes bf16 weights P_t to TMEM and adds to its
// row sum.  One exponential in four goes through a polynomial on the FMA pipe (d = 64).
//
// TMEM columns (NT = 2): S_A 0, S_B 128, O_A 256, O_B 256+d, and for d = 64 P_A 384, P_B 448; at
// d = 128 TMEM is full and P_t overlays the first 64 columns of S_t, so S_t(j+1) is issued behind
// O_t += P_t(j) V_j instead of ahead of it, and the two tiles take strict turns at the exponentials.
// Every wait is bounded (see tc_common.cuh); on expiry the CTA aborts cleanly and reports a code.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include <type_traits>

#include "flat_internal.cuh"
#include "ptx_sm100.cuh"
#include "tc_common.cuh"

namespace flat {

using namespace ptx;
using namespace tc;


namespace {

constexpr int BM = 128;              // rows per query tile (two tiles per CTA)
constexpr int BN = 128;              // keys per step
constexpr int PASS_AT_CHUNK = 2;                // the other tile gets its turn once this chunk's ex2 are issued (of chunks 0-3; measured on c4: 3 -> 1166, 2 -> 1187, 1 -> 995 TFLOP/s)
constexpr int POLY_LANE = 3;                    // element index mod 4 that uses ex2_poly; -1 = none
__host__ __device__ constexpr int merge_vecs(int d) { return d / 4 + 1; }   // (key split) 16-byte vectors per row of a partial result: d outputs, then (m, l)
constexpr float OVERFLOW_SUM = 1.0995116e12f;   // 2^40: a tile row sum beyond this means m_ref is stale

// BT: the bias tile of every (tile, step) is staged through shared memory by TMA (two stages per query tile)
// KHL (the two warpgroups of a CTA on alternate key tiles of ONE query tile, see the kernel's KH): every key tile has one
// consumer, the warpgroup of its parity, so the ring depths must be even -- stage g % depth then always belongs to
// the same warpgroup and a parity wait on its barrier is unambiguous.  (With three stages a stage alternates between
// the two consumers, each of which always waits for the SAME parity of its barrier, and a warpgroup that had run
// ahead could take the completion of its previous fill for that of the next one: wrong keys, then a stuck ring.
// Seen as rare wrong rows and time-outs on masked batches.)  1: four K and four V stages; 2: four and two (the
// sixteen-CTA cluster's receive buffer leaves no room for more).
template <int D, int NT, bool BT = false, int KHL = 0> struct L2 {
    static constexpr bool ALIAS = (D == 128);            // P overlays S
    static constexpr int KS = KHL ? 4 : (NT == 1 || BT) ? 2 : (D == 64) ? 3 : 2;   // K ring depth
    static constexpr int VS = KHL == 2 ? 2 : KS;         // V ring depth
    static constexpr int THREADS = 128 * NT + 128;       // NT softmax warpgroups + {TMA, NT MMA issuers, idle}
    static constexpr int SOFT_WARPS = 4 * NT;
    static constexpr uint32_t TMEM_COLS = (NT == 2) ? 512 : 256;
    static constexpr int Q_BYTES = BM * D * 2;           // one query tile
    static constexpr int KV_BYTES = BN * D * 2;
    static constexpr int BS = 2;                         // bias ring depth per query tile
    static constexpr int BIAS_BYTES = BM * BN * 2;       // one 128 x 128 bf16 tile: two panels of 128 rows x 128 bytes
    static constexpr int BIAS_OFF = NT * Q_BYTES + (KS + VS) * KV_BYTES;
    static constexpr int TILE_BYTES = BIAS_OFF + (BT ? NT * BS * BIAS_BYTES : 0);
    static constexpr int SMEM_BYTES = TILE_BYTES + 512 + 1024;
    __host__ __device__ static constexpr uint32_t S_COL(int t) { return 128u * t; }
    __host__ __device__ static constexpr uint32_t O_COL(int t) { return 128u * NT + D * t; }
    __host__ __device__ static constexpr uint32_t P_COL(int t) { return ALIAS ? 128u * t : 128u * NT + D * NT + 64u * t; }
    // barrier indices
    static constexpr int Q_FULL = 0;                     // [NT]
    static constexpr int K_FULL = NT, K_EMPTY = K_FULL + KS;
    static constexpr int V_FULL = K_EMPTY + KS, V_EMPTY = V_FULL + VS;
    static constexpr int S_FULL = V_EMPTY + VS;          // [NT]
    static constexpr int S_FREE = S_FULL + NT, P_FULL = S_FREE + NT, PV_DONE = P_FULL + NT;
    static constexpr int TURN = PV_DONE + NT;            // [2][4]: per warp pair, "tile t may run its exponentials"
    static constexpr int MERGE_BAR = TURN + 8;           // (key split over a cluster) partial results of the other CTAs have arrived
    static constexpr int B_FULL = MERGE_BAR + 1, B_EMPTY = B_FULL + NT * BS;   // (BT) [NT][BS]
    static constexpr int NUM_BARS = BT ? B_EMPTY + NT * BS : MERGE_BAR + 1;
    // rows of partial results a CTA of a CS-way split receives: CS - 1 senders x 128 / CS rows it owns
    __host__ __device__ static constexpr int merge_bytes(int cs) { return cs > 1 ? (cs - 1) * (128 / cs) * merge_vecs(D) * 16 : 0; }
    // Strict alternation of the two tiles' exponential phases.  At d = 128 the chain of a tile is
    // softmax -> (O += P V, next S) -> softmax with nothing to overlap inside the tile, so the tiles
    // must interleave: one computes exponentials while the other's MMAs run.  Left to themselves
    // they fall into lockstep and the phases add up instead.
    static constexpr bool TURNS = (NT == 2) && (D == 128);
};

__device__ __forceinline__ float row_max(const uint32_t (&s)[128]) {
    float e0 = __uint_as_float(s[0]), e1 = __uint_as_float(s[1]), e2 = __uint_as_float(s[2]), e3 = __uint_as_float(s[3]);
#pragma unroll
    for (int i = 4; i < 124; i += 8) {
        e0 = max3(e0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        e1 = max3(e1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        e2 = max3(e2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        e3 = max3(e3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
    }
    e0 = max3(e0, __uint_as_float(s[124]), __uint_as_float(s[125]));
    e1 = max3(e1, __uint_as_float(s[126]), __uint_as_float(s[127]));
    return fmaxf(fmaxf(e0, e1), fmaxf(e2, e3));
}
__device__ __forceinline__ float row_min(const uint32_t (&s)[128]) {
    float e0 = __uint_as_float(s[0]), e1 = __uint_as_float(s[1]), e2 = __uint_as_float(s[2]), e3 = __uint_as_float(s[3]);
#pragma unroll
    for (int i = 4; i < 124; i += 8) {
        e0 = min3(e0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        e1 = min3(e1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        e2 = min3(e2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        e3 = min3(e3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
    }
    e0 = min3(e0, __uint_as_float(s[124]), __uint_as_float(s[125]));
    e1 = min3(e1, __uint_as_float(s[126]), __uint_as_float(s[127]));
    return fminf(fminf(e0, e1), fminf(e2, e3));
}

// p_i = 2^(s_i * scale + neg_m) for one row of 128 logits; stores bf16(p) to 64 TMEM columns at
// `p_addr` and returns the fp32 sum of the unrounded p.  TAIL: only the first `nvalid` columns
// take part, the rest get p = 0 (this also removes the NaN of inf * 0 when scale == 0).
template <bool TAIL, bool POLY, typename BeforeFirstStore, typename AfterLastExp>
__device__ __forceinline__ float exp_store(const uint32_t (&s)[128], float scale_log2e, float neg_m, uint32_t p_addr,
                                           int nvalid, BeforeFirstStore&& before_first_store,
                                           AfterLastExp&& after_last_exp) {
    // Four chunks of 32 logits.  Within a chunk all FFMAs come first, then all exponentials, then
    // the sums and the bf16 packing, so that consecutive ex2 never wait on a neighbour.  The
    // logits s[] are left intact (a stale reference maximum may force a second pass over them).
    // The first chunk's weights are held in registers until the second chunk is done:
    // `before_first_store` (the wait for the P buffer to be free) then runs with a third of the
    // row already computed, late enough for the previous tile's O += P V to have finished.
    // Scale/shift and the row sums run on packed pairs (fma / add .f32x2: half the issue slots).
    uint64_t lsum0 = 0ull, lsum1 = 0ull;             // (l0, l1) and (l2, l3)
    const uint64_t scale2 = pack2(scale_log2e, scale_log2e), neg_m2 = pack2(neg_m, neg_m);
    uint32_t pk0[16];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint32_t pk[16];
        float p[32];
#pragma unroll
        for (int i = 0; i < 32; i += 2)
            unpack2(fma2(pack2(__uint_as_float(s[c * 32 + i]), __uint_as_float(s[c * 32 + i + 1])), scale2, neg_m2),
                    p[i], p[i + 1]);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            // One element in four takes the polynomial route (FMA pipe) to unload the ex2 unit,
            // the binding pipe at d = 64; the careful/tail pass keeps to ex2 throughout, and so do
            // the tiles that take turns (POLY off): a warp running alone is short of issue slots,
            // not of ex2 throughput.
            p[i] = (!TAIL && POLY && (i & 3) == POLY_LANE) ? ex2_poly(p[i]) : ex2_approx(p[i]);
            if (TAIL && c * 32 + i >= nvalid) p[i] = 0.f;
        }
        if (c == PASS_AT_CHUNK) after_last_exp();       // most ex2 of the row have been issued
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            lsum0 = add2(lsum0, pack2(p[i], p[i + 1]));
            lsum1 = add2(lsum1, pack2(p[i + 2], p[i + 3]));
            pk[i / 2] = pack_bf16x2(p[i], p[i + 1]);
            pk[i / 2 + 1] = pack_bf16x2(p[i + 2], p[i + 3]);
        }
        if (c == 0) {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk0[i] = pk[i];
        } else {
            if (c == 1) { before_first_store(); tmem_st_x16(p_addr, pk0); }
            tmem_st_x16(p_addr + c * 16, pk);
        }
    }
    float l0, l1, l2, l3;
    unpack2(lsum0, l0, l1);
    unpack2(lsum1, l2, l3);
    return (l0 + l1) + (l2 + l3);
}

// VL: packed variable-length batches.  Q, O are [total_q, H, d], K, V [total_k, H, d]; sequence s owns
// tokens cu_q[s] .. cu_q[s+1] - 1 of Q and cu_k[s] .. cu_k[s+1] - 1 of K, V; the tensor maps view the
// packed tensors as {d, H, tokens}; blockIdx.y = sequence * H + head, blockIdx.x = slab of the
// sequence's rows (a CTA past the end of its sequence leaves at once); the causal offset is that of
// the sequence; valid_len is unused.
// BIAS: a separate instantiation that adds a bias tensor to the scaled logits (dense batches): the softmax
// thread fetches its row's 128 values of the step straight from device memory -- a bf16 bias adds
// 2 B H Nq Nk bytes of traffic, four times |Q|+|K|+|V|+|O| on a 4096 x 4096, d = 64 problem.
// SPARSE (one tile per CTA): pruned attention.  A byte map over 128 x 128 blocks of the logit matrix says
// which key tiles the CTA's query tile attends; the CTA compacts its row of the map into a list in shared
// memory and every role walks that list instead of 0, 1, 2, ...: pruned key tiles are neither loaded nor
// multiplied.
// CS > 1 (one tile per CTA, dense): the keys of a query tile are split over the CS CTAs of a thread-block
// cluster (2, 4 or 8) -- for launches that would leave most SMs empty.  Each CTA runs the pipeline over its share of
// the key tiles and ends with a partial (m, l, O) per row; rank r owns rows [128 r / CS, 128 (r + 1) / CS): the other
// ranks store their partials for those rows into r's shared memory (st.shared::cluster, lanes of a warp writing
// contiguous bytes) and arrive on r's mbarrier, and the owner merges them with the split-softmax identity and writes
// the rows.  Plain remote stores only.
// BIAS = 2: the same with the bias tile of each step staged through shared memory by TMA (bf16, 16-byte aligned
// rows, d = 64): the rows then arrive coalesced and a softmax thread reads its 256 bytes from shared memory; with a
// bias shared by all batches the grid runs the batches of a head next to each other, so that its slice stays in L2.
// KH (two warpgroups, ONE query tile, d = 64, dense): a short launch waits for one CTA's chain of key steps, and a
// step is one warp per scheduler working through 128 exponentials per row.  With KH the CTA's two softmax warpgroups
// (and their two MMA issuers, logit / weight / output columns) take the even and the odd key tiles of the same 128
// query rows, each with its own running (m_ref, l, O); at the end the second warpgroup leaves its rows in shared
// memory and the first merges them (the split-softmax identity again) before the ordinary epilogue or the cluster
// exchange.  The chain is half as long and two warps per scheduler share the exponent unit.
template <int D, int NT, bool VL = false, int BIAS = 0, bool SPARSE = false, int CS = 1, bool KH = false>
__global__ void __launch_bounds__(128 * NT + 128, NT == 1 ? 2 : 1)
fused_tc2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, int H, int Nq, int Nk,
                 float scale_log2e, const int32_t* __restrict__ valid_len, int coff, int32_t* status,
                 const int32_t* __restrict__ cu_q = nullptr, const int32_t* __restrict__ cu_k = nullptr,
                 float* __restrict__ lse = nullptr, BiasArg bias = BiasArg{nullptr, 0, 0, 0, 0},
                 const uint8_t* __restrict__ block_mask = nullptr, long long bmask_sb = 0, long long bmask_sh = 0,
                 const __grid_constant__ CUtensorMap tmBias = CUtensorMap{}) {
    using LY = L2<D, NT, BIAS == 2, KH ? (CS == 16 ? 2 : 1) : 0>;
    static_assert(BIAS != 2 || (NT == 2 && D == 64 && !VL && !SPARSE && CS == 1), "staged bias: the two-tile dense kernel, d = 64");
    static_assert(!SPARSE || (NT == 1 && !VL && !BIAS), "the pruning map is read by the one-tile dense kernel");
    static_assert(CS == 1 || ((NT == 1 || KH) && !VL && !BIAS && !SPARSE && (CS == 2 || CS == 4 || CS == 8 || CS == 16)), "key split: one-tile dense kernel");
    static_assert(!KH || (NT == 2 && D == 64 && !VL && !BIAS && !SPARSE), "key halves: two warpgroups on one dense d = 64 tile");
    constexpr int QT = KH ? 1 : NT;                      // query tiles of the CTA
    __shared__ uint16_t tile_list[SPARSE ? 1024 : 1];    // the kept key tiles of this query tile, ascending
    __shared__ int tile_count;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Qs = base;                                  // NT tiles
    uint8_t* Ks = Qs + NT * LY::Q_BYTES;                  // KS tiles
    uint8_t* Vs = Ks + LY::KS * LY::KV_BYTES;            // VS tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + LY::TILE_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + LY::NUM_BARS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float4* merge_buf = reinterpret_cast<float4*>(base + LY::TILE_BYTES + 512);   // (CS > 1) [CS - 1][d / 4 + 1][128 / CS]: lanes of a warp touch contiguous bytes
    float4* kh_buf = reinterpret_cast<float4*>(base + LY::TILE_BYTES + 512 + LY::merge_bytes(CS));   // (KH) [d / 4 + 1][128]: the second warpgroup's rows

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bh = blockIdx.y;
    if (BIAS == 2 && bias.sb == 0) {
        // a bias shared by the batches: y runs over the batches first, so that CTAs in flight share a head's slice
        const int nb = gridDim.y / H;
        bh = (blockIdx.y % nb) * H + blockIdx.y / nb;
    }
    const int crank = CS > 1 ? static_cast<int>(cluster_ctarank()) : 0;   // (cluster = CS consecutive CTAs along x)
    const int row0 = (blockIdx.x / CS) * (QT * BM);
    // Barriers and TMEM columns.  The one-tile dense kernels (short launches, where the gap between two kernels of a
    // stream is a good part of the time) do this before anything else and then let the next kernel of the stream
    // start its own set-up (griddepcontrol.launch_dependents) and wait for the previous one to finish
    // (griddepcontrol.wait) before the first access to device memory: launched with programmatic stream
    // serialization, consecutive kernels overlap one's tail with the other's prologue.
    constexpr bool PDL = ((NT == 1 || KH) && !VL && !SPARSE && !BIAS);
    auto setup = [&]() {
        if (threadIdx.x == LY::SOFT_WARPS * 32) {
            for (int i = 0; i < LY::NUM_BARS; ++i) {
                const bool by_softmax = (i >= LY::S_FREE && i < LY::PV_DONE) ||    // one arrival per softmax warp
                                        (BIAS == 2 && i >= LY::B_EMPTY);
                const bool by_issuers = (i >= LY::K_EMPTY && i < LY::V_FULL) || (i >= LY::V_EMPTY && i < LY::S_FULL);
                mbar_init(&bars[i], i == LY::MERGE_BAR ? (CS > 1 ? (CS - 1) * (CS <= 4 ? 128 / CS / 32 : 1) : 1) : by_softmax ? 4 : by_issuers ? (KH ? 1 : NT) : 1);   // (KH: a key tile is used by one warpgroup only)
            }
            *abort_flag = 0;
            fence_mbar_init();
        }
        if (warp == 0) { tmem_alloc(tmem_slot, LY::TMEM_COLS); tmem_relinquish(); }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    };
    if (PDL) {
        setup();
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    int n = Nk;
    int head = 0, q_tok0 = 0, k_tok0 = 0, q_rows = 0;    // (packed batches only)
    if (VL) {
        const int s = bh / H;
        head = bh - s * H;
        const int q0 = cu_q[s], ql = cu_q[s + 1] - q0, k0 = cu_k[s], kl = cu_k[s + 1] - k0;
        if (row0 >= ql) return;                          // (the whole CTA: nothing is set up yet)
        q_tok0 = q0 + row0; k_tok0 = k0; q_rows = ql - row0;
        n = kl < 0 ? 0 : kl;
        if (coff < (1 << 29)) coff = kl - ql;
    } else if (valid_len) { n = valid_len[bh / H]; n = n < 0 ? 0 : (n > Nk ? Nk : n); }
    {
        // Causal mask (coff = Nk - Nq; 2^30 = none): row r sees keys j < r + 1 + coff, so the CTA's
        // last row bounds the keys of all its rows.
        const long long lim = static_cast<long long>(row0) + QT * BM + coff;
        if (lim < n) n = lim < 0 ? 0 : static_cast<int>(lim);
    }
    int ntiles = (n + BN - 1) / BN;
    int tile0 = 0;                                       // first key tile of this CTA
    if (CS > 1) {
        const int per = (ntiles + CS - 1) / CS, left = ntiles - crank * per;
        tile0 = crank * per;
        ntiles = left < 0 ? 0 : (left > per ? per : left);
    }
    if (SPARSE && (threadIdx.x >> 5) == 1) {
        // warp 1 compacts the map's row (tiles below the key limit n only) into the list
        const uint8_t* mrow = block_mask + static_cast<long long>(bh / H) * bmask_sb + static_cast<long long>(bh % H) * bmask_sh +
                              static_cast<long long>(blockIdx.x) * ((Nk + BN - 1) / BN);
        const int ln = threadIdx.x & 31;
        int count = 0;
        for (int base = 0; base < ntiles; base += 32) {
            const int jj = base + ln;
            const bool keep = jj < ntiles && mrow[jj] != 0;
            const unsigned m = __ballot_sync(0xffffffffu, keep);
            if (keep) tile_list[count + __popc(m & ((1u << ln) - 1u))] = static_cast<uint16_t>(jj);
            count += __popc(m);
        }
        if (ln == 0) tile_count = count;
    }

    if (!PDL) setup();
    const uint32_t tmem = *tmem_slot;
    if (CS > 1) cluster_sync_all();                      // every CTA of the cluster has its barriers before anyone's first remote access
    if (SPARSE) ntiles = tile_count;
    // key tile of step j: the j-th kept one under a pruning map, else the j-th of this CTA's range
    auto tile_of = [&](int j) -> int { return SPARSE ? static_cast<int>(tile_list[j]) : tile0 + j; };

    if (warp >= LY::SOFT_WARPS) {
      if (NT == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
      else         asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");
      if (warp == LY::SOFT_WARPS) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0 && ntiles > 0) {
            prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
            bool ok = true;
            int k_issued = 0, v_issued = 0;
            auto load_k = [&](int j) {
                const int s = j % LY::KS;
                ok = bounded_wait(&bars[LY::K_EMPTY + s], ((j / LY::KS) & 1) ^ 1, abort_flag, status, 0x100 + s);
                if (!ok) return;
                mbar_arrive_expect_tx(&bars[LY::K_FULL + s], LY::KV_BYTES);
#pragma unroll
                for (int c = 0; c < D / 64; ++c)
                    tma_load_3d(Ks + s * LY::KV_BYTES + c * BN * 128, &tmK, &bars[LY::K_FULL + s], c * 64, VL ? head : tile_of(j) * BN,
                                VL ? k_tok0 + j * BN : bh);
                k_issued = j + 1;
            };
            auto load_v = [&](int j) {
                const int s = j % LY::VS;
                ok = bounded_wait(&bars[LY::V_EMPTY + s], ((j / LY::VS) & 1) ^ 1, abort_flag, status, 0x110 + s);
                if (!ok) return;
                mbar_arrive_expect_tx(&bars[LY::V_FULL + s], LY::KV_BYTES);
#pragma unroll
                for (int c = 0; c < D / 64; ++c)
                    tma_load_3d(Vs + s * LY::KV_BYTES + c * BN * 128, &tmV, &bars[LY::V_FULL + s], c * 64, VL ? head : tile_of(j) * BN,
                                VL ? k_tok0 + j * BN : bh);
                v_issued = j + 1;
            };
            int b_issued = 0;
            auto load_b = [&](int j) {                   // (BIAS == 2) the bias tiles of step j, one per query tile
                const int s = j % LY::BS;
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    if (!ok) return;
                    ok = bounded_wait(&bars[LY::B_EMPTY + t * LY::BS + s], ((j / LY::BS) & 1) ^ 1, abort_flag, status, 0x120 + t);
                    if (!ok) return;
                    uint8_t* dst = base + LY::BIAS_OFF + (t * LY::BS + s) * LY::BIAS_BYTES;
                    mbar_arrive_expect_tx(&bars[LY::B_FULL + t * LY::BS + s], LY::BIAS_BYTES);
#pragma unroll
                    for (int c = 0; c < 2; ++c)
                        tma_load_4d(dst + c * BM * 128, &tmBias, &bars[LY::B_FULL + t * LY::BS + s], j * BN + c * 64, row0 + t * BM,
                                    bias.sh ? bh % H : 0, bias.sb ? bh / H : 0);
                }
                b_issued = j + 1;
            };
            if (BIAS == 2) prefetch_tensormap(&tmBias);
            mbar_arrive_expect_tx(&bars[LY::Q_FULL + 0], LY::Q_BYTES);
#pragma unroll
            for (int c = 0; c < D / 64; ++c)
                tma_load_3d(Qs + c * BM * 128, &tmQ, &bars[LY::Q_FULL + 0], c * 64, VL ? head : row0, VL ? q_tok0 : bh);
            load_k(0);
            if (BIAS == 2) load_b(0);
            if (NT == 2) {
                mbar_arrive_expect_tx(&bars[LY::Q_FULL + NT - 1], LY::Q_BYTES);
#pragma unroll
                for (int c = 0; c < D / 64; ++c)
                    tma_load_3d(Qs + (NT - 1) * LY::Q_BYTES + c * BM * 128, &tmQ, &bars[LY::Q_FULL + NT - 1], c * 64,
                                VL ? head : row0 + (KH ? 0 : BM), VL ? q_tok0 + BM : bh);   // (KH: the same rows again)
            }
            for (int j = 0; j < ntiles && ok; ++j) {
                if (j + 1 < ntiles) load_k(j + 1);
                if (ok) load_v(j);
                if (BIAS == 2 && ok && j + 1 < ntiles) load_b(j + 1);
            }
            if (!ok) {
                if (BIAS == 2)
                    for (int j = b_issued > LY::BS ? b_issued - LY::BS : 0; j < b_issued; ++j)
                        for (int t = 0; t < NT; ++t) drain_wait(&bars[LY::B_FULL + t * LY::BS + j % LY::BS], (j / LY::BS) & 1);
                drain_wait(&bars[LY::Q_FULL + 0], 0);
                if (NT == 2) drain_wait(&bars[LY::Q_FULL + NT - 1], 0);
                for (int j = k_issued > LY::KS ? k_issued - LY::KS : 0; j < k_issued; ++j)
                    drain_wait(&bars[LY::K_FULL + j % LY::KS], (j / LY::KS) & 1);
                for (int j = v_issued > LY::VS ? v_issued - LY::VS : 0; j < v_issued; ++j)
                    drain_wait(&bars[LY::V_FULL + j % LY::VS], (j / LY::VS) & 1);
            }
        }
      } else if (warp <= LY::SOFT_WARPS + NT) {
        // ------------------------------------------------------------ MMA issuer of tile t
        // The whole warp runs this loop (uniform control flow); one elected lane issues.
        const int t = warp - LY::SOFT_WARPS - 1;
        // (KH: this warpgroup's key tiles are every second one of the CTA's sequence; the rings are indexed with
        // the position in that sequence, the tile's own barriers with the count of its own steps)
        const int nt_t = KH ? (ntiles - t + 1) / 2 : ntiles;
        auto gi = [&](int j) -> int { return KH ? 2 * j + t : j; };
        if (nt_t > 0) {
            constexpr uint32_t IDESC_S = make_idesc_bf16(BM, BN, 0, 0);
            constexpr uint32_t IDESC_PV = make_idesc_bf16(BM, D, 0, 1);
            const uint64_t q_desc = make_smem_desc_sw128(smem_u32(Qs) + t * LY::Q_BYTES, 16, 1024);
            const uint64_t k_desc = make_smem_desc_sw128(smem_u32(Ks), 16, 1024);
            const uint64_t v_desc = make_smem_desc_sw128(smem_u32(Vs), BN * 128, 1024);
            const uint32_t s_tmem = tmem + LY::S_COL(t), o_tmem = tmem + LY::O_COL(t), p_tmem = tmem + LY::P_COL(t);
            bool ok = true;
            auto wait = [&](int bar, uint32_t parity, int code) {
                if (ok) ok = __all_sync(0xffffffffu, bounded_wait(&bars[bar], parity, abort_flag, status, code));
                if (ok) tc_fence_after();
            };
            auto issue_s = [&](int j) {                  // S_t = Q_t K_j^T, then release the K stage
                const int ks = gi(j) % LY::KS;
                if (elect_one()) {
                    const uint64_t kd = k_desc + static_cast<uint64_t>((ks * LY::KV_BYTES) >> 4);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint64_t off = static_cast<uint64_t>(((k / 4) * (BM * 128) + (k % 4) * 32) >> 4);
                        mma_ss(s_tmem, q_desc + off, kd + off, IDESC_S, k > 0);
                    }
                    tc_commit(&bars[LY::S_FULL + t]);
                    tc_commit(&bars[LY::K_EMPTY + ks]);
                }
                __syncwarp();
            };
            auto issue_pv = [&](int j) {                 // O_t += P_t V_j, then release the V stage
                const int vs = gi(j) % LY::VS;
                if (elect_one()) {
                    const uint64_t vd = v_desc + static_cast<uint64_t>((vs * LY::KV_BYTES) >> 4);
#pragma unroll
                    for (int k = 0; k < BN / 16; ++k)
                        mma_ts(o_tmem, p_tmem + k * 8, vd + static_cast<uint64_t>((k * 2048) >> 4), IDESC_PV,
                               (j > 0 || k > 0));
                    tc_commit(&bars[LY::PV_DONE + t]);
                    tc_commit(&bars[LY::V_EMPTY + vs]);
                }
                __syncwarp();
            };
            wait(LY::Q_FULL + t, 0, 0x200 + t);
            wait(LY::K_FULL + gi(0) % LY::KS, (gi(0) / LY::KS) & 1, 0x202);
            if (ok) issue_s(0);
            for (int j = 0; j < nt_t && ok; ++j) {
                const bool more = j + 1 < nt_t;
                const int ks = gi(j + 1) % LY::KS, vs = gi(j) % LY::VS;
                const uint32_t kph = (gi(j + 1) / LY::KS) & 1, vph = (gi(j) / LY::VS) & 1;
                if (!LY::ALIAS && more) {
                    // P has columns of its own: the next S_t only needs the softmax to have taken S_t(j)
                    wait(LY::K_FULL + ks, kph, 0x210);
                    wait(LY::S_FREE + t, j & 1, 0x211);
                    if (ok) issue_s(j + 1);
                }
                wait(LY::V_FULL + vs, vph, 0x220);
                // (P overlays S: the next key tile's barrier is checked here, while the softmax still runs, so that
                // the next S_t can go straight behind the MMA that reads P_t(j): a barrier check costs about 150
                // cycles of the tile's chain even when the tile has long arrived)
                if (LY::ALIAS && more) wait(LY::K_FULL + ks, kph, 0x230);
                wait(LY::P_FULL + t, j & 1, 0x221);
                if (ok) issue_pv(j);
                if (LY::ALIAS && more && ok) issue_s(j + 1);
            }
        }
      }
    } else {
        // ------------------------------------------------------------ softmax + epilogue (warps 0-7)
        if (NT == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        else         asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int t = warp >> 2;                         // query tile of this warpgroup (KH: its half of the key tiles)
        const int row = row0 + (KH ? 0 : t * BM) + (warp & 3) * 32 + lane;
        const int nt_t = KH ? (ntiles - t + 1) / 2 : ntiles;
        auto gi = [&](int j) -> int { return KH ? 2 * j + t : j; };
        const uint32_t tl = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        // (with a bias the logits are rescaled and shifted as they arrive, and the step goes on with scale 1)
        const float sc = BIAS ? 1.f : scale_log2e;
        const bool neg_scale = BIAS ? false : scale_log2e < 0.f;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        // keys this thread's row sees; lane 0 has the shortest row of the warp
        const long long rlim = static_cast<long long>(row) + 1 + coff;
        const int nrow = rlim < n ? (rlim < 0 ? 0 : static_cast<int>(rlim)) : n;
        const int nrow_min = __shfl_sync(0xffffffffu, nrow, 0);
        if (LY::TURNS && t == 1 && lane == 0) mbar_arrive(&bars[LY::TURN + (warp & 3)]);   // tile A goes first
        for (int j = 0; j < nt_t; ++j) {
            // (bias, the common case of an aligned bf16 tensor: the row's 128 values of this step are fetched
            // before the wait for the logits, so that the two latencies overlap)
            uint32_t bpk[BIAS == 1 ? 64 : 1];
            bool bias_ready = false;
            if (BIAS == 1) {
                if (bias.vec && !bias.f32 && row < Nq && (j + 1) * BN <= Nk) {
                    const uint4* g = reinterpret_cast<const uint4*>(
                        static_cast<const __nv_bfloat16*>(bias.p) + static_cast<long long>(bh / H) * bias.sb +
                        static_cast<long long>(bh % H) * bias.sh + static_cast<long long>(row) * Nk + j * BN);
#pragma unroll
                    for (int v = 0; v < 16; ++v) {
                        const uint4 w = g[v];
                        bpk[4 * v] = w.x; bpk[4 * v + 1] = w.y; bpk[4 * v + 2] = w.z; bpk[4 * v + 3] = w.w;
                    }
                    bias_ready = true;
                }
            }
            ok = bounded_wait(&bars[LY::S_FULL + t], j & 1, abort_flag, status, 0x300 + t);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t s[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_x32(tl + LY::S_COL(t) + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[LY::S_FREE + t]);   // S_t may be overwritten (d = 64: by the next S_t)

            const int col0 = tile_of(gi(j)) * BN;
            if (BIAS == 2) {
                // x = s * scale * log2(e) + bias * log2(e): the thread's row of the staged tile (two swizzled panels)
                const int bs = j % LY::BS, rt = (warp & 3) * 32 + lane;
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::B_FULL + t * LY::BS + bs], (j / LY::BS) & 1, abort_flag,
                                                         status, 0x360 + t));
                if (!ok) break;
                const uint8_t* brow = base + LY::BIAS_OFF + (t * LY::BS + bs) * LY::BIAS_BYTES + rt * 128;
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const uint4 w = *reinterpret_cast<const uint4*>(brow + (c >> 3) * (BM * 128) + (((c & 7) ^ (rt & 7)) << 4));
                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        s[c * 8 + 2 * e] = __float_as_uint(fmaf(__uint_as_float(s[c * 8 + 2 * e]), scale_log2e,
                                                                __uint_as_float(ww[e] << 16) * 1.4426950408889634f));
                        s[c * 8 + 2 * e + 1] = __float_as_uint(fmaf(__uint_as_float(s[c * 8 + 2 * e + 1]), scale_log2e,
                                                                    __uint_as_float(ww[e] & 0xffff0000u) * 1.4426950408889634f));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[LY::B_EMPTY + t * LY::BS + bs]);
            } else if (BIAS) {
                // x = s * scale * log2(e) + bias * log2(e); a row past the end and columns past Nk read nothing
                const long long at = static_cast<long long>(bh / H) * bias.sb + static_cast<long long>(bh % H) * bias.sh +
                                     static_cast<long long>(row) * Nk + col0;
                const bool in_rows = row < Nq;
                if (bias_ready) {
#pragma unroll
                    for (int i = 0; i < 64; ++i) {
                        s[2 * i] = __float_as_uint(fmaf(__uint_as_float(s[2 * i]), scale_log2e,
                                                        __uint_as_float(bpk[i] << 16) * 1.4426950408889634f));
                        s[2 * i + 1] = __float_as_uint(fmaf(__uint_as_float(s[2 * i + 1]), scale_log2e,
                                                            __uint_as_float(bpk[i] & 0xffff0000u) * 1.4426950408889634f));
                    }
                } else if (bias.vec && in_rows && col0 + BN <= Nk) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {        // sixteen columns at a time (few registers live)
                        float bv[16];
                        if (bias.f32) {
                            const float4* g = reinterpret_cast<const float4*>(static_cast<const float*>(bias.p) + at + c * 16);
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                const float4 w = g[v];
                                bv[4 * v] = w.x; bv[4 * v + 1] = w.y; bv[4 * v + 2] = w.z; bv[4 * v + 3] = w.w;
                            }
                        } else {
                            const uint4* g = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(bias.p) + at + c * 16);
#pragma unroll
                            for (int v = 0; v < 2; ++v) {
                                const uint4 w = g[v];
                                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    bv[8 * v + 2 * e] = __uint_as_float(ww[e] << 16);
                                    bv[8 * v + 2 * e + 1] = __uint_as_float(ww[e] & 0xffff0000u);
                                }
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            s[c * 16 + i] = __float_as_uint(fmaf(__uint_as_float(s[c * 16 + i]), scale_log2e, bv[i] * 1.4426950408889634f));
                    }
                } else {
#pragma unroll                                           // (fully: the logits must stay in registers)
                    for (int i = 0; i < 128; ++i) {
                        float bvi = 0.f;
                        if (in_rows && col0 + i < Nk)
                            bvi = bias.f32 ? static_cast<const float*>(bias.p)[at + i]
                                           : __bfloat162float(static_cast<const __nv_bfloat16*>(bias.p)[at + i]);
                        s[i] = __float_as_uint(fmaf(__uint_as_float(s[i]), scale_log2e, bvi * 1.4426950408889634f));
                    }
                }
            }
            const bool tail = col0 + BN > nrow_min;      // (warp-uniform) some row has masked keys in this step
            const int nvalid = nrow > col0 ? (nrow - col0 < BN ? nrow - col0 : BN) : 0;   // per row
            if (tail) {
                const uint32_t excl = __float_as_uint(neg_scale ? INFINITY : -INFINITY);
#pragma unroll
                for (int i = 0; i < 128; ++i) if (i >= nvalid) s[i] = excl;
            }
            // At d = 64 P_t is a single buffer: O_t += P_t(j-1) V must have consumed it before the
            // first store of P_t(j).  The wait sits inside the exponential pipeline (see exp_store).
            bool pv_waited = LY::ALIAS || j == 0;
            auto wait_p_free = [&]() {
                if (!pv_waited) {
                    ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::PV_DONE + t], (j - 1) & 1, abort_flag,
                                                             status, 0x320 + t));
                    pv_waited = true;
                }
            };
            bool turn_passed = !LY::TURNS;
            auto pass_turn = [&]() {
                if (!turn_passed) {
                    turn_passed = true;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars[LY::TURN + (t ^ 1) * 4 + (warp & 3)]);
                }
            };
            if (LY::TURNS) {
                ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::TURN + t * 4 + (warp & 3)], j & 1, abort_flag,
                                                         status, 0x340 + t));
                if (!ok) break;
            }
            // p = 2^(scale*s - m_ref); row sum in fp32 from the unrounded p; P rounded to bf16.
            // Any reference m_ref gives the exact softmax, so the common case reuses the one in
            // hand and takes no row maximum at all; a row sum beyond 2^40 (or inf/NaN) shows that
            // the reference fell too far behind, and the tile is then redone the careful way.
            bool careful = (j == 0) || tail;
            float lt = 0.f;
            if (!careful) {
                lt = exp_store<false, !LY::TURNS>(s, sc, -m_ref, tl + LY::P_COL(t), BN, wait_p_free, pass_turn);
                if (!ok) break;                           // (a failed wait means the stores went nowhere useful)
                careful = __any_sync(0xffffffffu, !(lt <= OVERFLOW_SUM));
            }
            if (careful) {
                // (a row with no valid key in this step -- causal mask -- contributes no maximum)
                const float mx = nvalid > 0 ? (neg_scale ? row_min(s) : row_max(s)) * sc : -INFINITY;
                if (__any_sync(0xffffffffu, mx > m_ref + RESCALE_THRESHOLD)) {
                    const float m_new = fmaxf(m_ref, mx);
                    // 0 on the first tile; a row that has not seen a valid key yet keeps l = 0
                    const float alpha = m_new == -INFINITY ? 1.f : ex2_approx(m_ref - m_new);
                    l *= alpha;
                    if (j > 0) {
                        ok = __all_sync(0xffffffffu, bounded_wait(&bars[LY::PV_DONE + t], (j - 1) & 1, abort_flag,
                                                                 status, 0x310 + t));
                        if (!ok) break;
                        pv_waited = true;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t r[32];
                            tmem_ld_x32(tl + LY::O_COL(t) + c * 32, r);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                            tmem_st_x32(tl + LY::O_COL(t) + c * 32, r);
                        }
                    }
                    m_ref = m_new;
                }
                // (a row whose every pair so far was switched off by a -inf bias still has no reference:
                // 0 then stands in, so that its weights come out as 2^-inf = 0 and not as NaN)
                lt = exp_store<true, false>(s, sc, (BIAS && m_ref == -INFINITY) ? 0.f : -m_ref, tl + LY::P_COL(t), nvalid,
                                            wait_p_free, pass_turn);
                if (!ok) break;
            }
            l += lt;
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[LY::P_FULL + t]);
        }
        if (ok && nt_t > 0) {
            ok = bounded_wait(&bars[LY::PV_DONE + t], (nt_t - 1) & 1, abort_flag, status, 0x330 + t);
            ok = __all_sync(0xffffffffu, ok);
        }
        if constexpr (CS > 1 || KH) {
            // ---- partial (m, l, O) rows: merged inside the CTA (KH), exchanged inside the cluster (CS > 1), written
            constexpr int RP = 128 / CS;                  // rows owned per rank: whole warps, or half a warp at CS = 8
            constexpr int GRP = RP < 32 ? RP : 32;        // lanes of a warp that share an owner
            const int tr = (warp & 3) * 32 + lane, owner = tr / RP;
            float o[D];
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                if (ok && nt_t > 0) {
                    tmem_ld_x32(tl + LY::O_COL(t) + c * 32, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;      // no key tile in this share
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) o[c * 32 + i] = __uint_as_float(r[i]);
            }
            if (!ok) l = __int_as_float(0x7fc00000);     // (a share that gave up poisons the rows it took part in)
            // (m, l, O) of two shares of a row's keys: m = max, l = sum of l_i 2^(m_i - m), O likewise
            auto merge_row = [&](const float4* src, int stride) {
                const float mq = src[stride * (D / 4)].x, lq = src[stride * (D / 4)].y;
                const float mt = fmaxf(m_ref, mq), mu = mt == -INFINITY ? 0.f : mt;
                const float a = ex2_approx(m_ref - mu), b = ex2_approx(mq - mu);
                l = l * a + lq * b;
                m_ref = mt;
#pragma unroll
                for (int v = 0; v < D / 4; ++v) {
                    const float4 w = src[stride * v];
                    o[4 * v] = o[4 * v] * a + w.x * b;         o[4 * v + 1] = o[4 * v + 1] * a + w.y * b;
                    o[4 * v + 2] = o[4 * v + 2] * a + w.z * b; o[4 * v + 3] = o[4 * v + 3] * a + w.w * b;
                }
            };
            bool writer = true;
            if constexpr (KH) {
                // the second warpgroup hands its rows to the first through shared memory (lanes of a warp write
                // contiguous 16-byte vectors) and is done; a named barrier of the eight softmax warps in between
                if (t == 1) {
#pragma unroll
                    for (int v = 0; v < D / 4; ++v) kh_buf[v * 128 + tr] = make_float4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
                    kh_buf[(D / 4) * 128 + tr] = make_float4(m_ref, l, 0.f, 0.f);
                }
                asm volatile("bar.sync 2, 256;" ::: "memory");
                if (t == 1) writer = false;
                else merge_row(kh_buf + tr, 128);
            }
            if constexpr (CS > 1) {
                if (writer) {                             // (warp-uniform)
                    if (owner != crank) {
                        const int slot = (crank - owner - 1 + CS) % CS;
                        const uint32_t dst = mapa_shared(smem_u32(merge_buf + slot * merge_vecs(D) * RP + tr % RP), owner);
#pragma unroll
                        for (int v = 0; v < D / 4; ++v) st_cluster_v4(dst + 16 * RP * v, o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
                        st_cluster_v2(dst + 16 * RP * (D / 4), m_ref, l);
                    }
                    // one arrival per group of lanes with the same owner: the warp barrier orders the lanes' stores
                    // before the first lane's release
                    __syncwarp();
                    if (owner != crank && lane % GRP == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&bars[LY::MERGE_BAR]), owner));
                    writer = owner == crank;
                    if (writer) {
                        // An owner must not leave before its senders have stored (a remote store into the shared
                        // memory of a CTA that has left is a fault).  Every sender stores and arrives whatever
                        // happened to it: its roles give up at their first wait that runs out (WAIT_CYCLES) and go
                        // straight to the exchange, and the CTAs of a cluster start together -- so the owner waits
                        // four times as long as any sender can take before it gives up itself.
                        const long long t0 = clock64();
                        while (!mbar_try_wait_cluster(&bars[LY::MERGE_BAR], 0)) {
                            if (clock64() - t0 > 4 * WAIT_CYCLES) {
                                writer = false;
                                if (status) atomicExch(status, 0x350);
                                break;
                            }
                        }
                    }
                    if (writer) {
#pragma unroll
                        for (int q = 0; q < CS - 1; ++q) merge_row(merge_buf + q * merge_vecs(D) * RP + tr % RP, RP);
                    }
                }
            }
            if (writer && row < Nq) {
                const float inv = l > 0.f ? 1.f / l : (l == l ? 0.f : l);
                if (lse) lse[static_cast<int64_t>(bh) * Nq + row] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
                __nv_bfloat16* orow = O + (static_cast<int64_t>(bh) * Nq + row) * D;
#pragma unroll
                for (int v = 0; v < D / 8; ++v) {
                    uint4 w;
                    w.x = pack_bf16x2(o[8 * v + 0] * inv, o[8 * v + 1] * inv);
                    w.y = pack_bf16x2(o[8 * v + 2] * inv, o[8 * v + 3] * inv);
                    w.z = pack_bf16x2(o[8 * v + 4] * inv, o[8 * v + 5] * inv);
                    w.w = pack_bf16x2(o[8 * v + 6] * inv, o[8 * v + 7] * inv);
                    *reinterpret_cast<uint4*>(orow + v * 8) = w;
                }
            }
        } else
        if (ok) {
            const float inv = l > 0.f ? 1.f / l : 0.f;
            // (dense batches only) log of the row's sum of exponentials; m_ref and the exponents are in base-2 units
            if (!VL && lse && row < Nq)
                lse[static_cast<int64_t>(bh) * Nq + row] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            tc_fence_after();
            __nv_bfloat16* orow = VL ? O + ((static_cast<int64_t>(q_tok0) + (row - row0)) * H + head) * D
                                     : O + (static_cast<int64_t>(bh) * Nq + row) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                if (ntiles > 0) {
                    tmem_ld_x32(tl + LY::O_COL(t) + c * 32, r);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;      // no valid key: O = 0
                }
                if (VL ? row - row0 < q_rows : row < Nq) {
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
    if (warp == 0) tmem_dealloc(tmem, LY::TMEM_COLS);
}

// The bias [B or 1, H or 1, Nq, Nk] bf16 as a 4-D tensor {Nk, Nq, heads, batches} with boxes of 64 columns x 128
// rows (one 128-byte-swizzled panel); a broadcast axis has extent 1 and is always read at coordinate 0.
bool make_bias_map(CUtensorMap* m, const Problem& p) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    const cuuint64_t rowb = static_cast<cuuint64_t>(p.Nk) * 2, slice = static_cast<cuuint64_t>(p.Nq) * rowb;
    const cuuint64_t sh = p.bias_sh ? static_cast<cuuint64_t>(p.bias_sh) * 2 : slice;
    const cuuint64_t hb = p.bias_sh ? p.H : 1, bb = p.bias_sb ? p.B : 1;
    const cuuint64_t sb = p.bias_sb ? static_cast<cuuint64_t>(p.bias_sb) * 2 : sh * hb;
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(p.Nk), static_cast<cuuint64_t>(p.Nq), hb, bb};
    cuuint64_t strides[3] = {rowb, sh, sb};
    cuuint32_t box[4] = {64, static_cast<cuuint32_t>(BM), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(p.bias), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Clusters of sixteen CTAs are more than the portable cluster size: the kernel must opt in, and the device must be
// able to hold such a cluster at all (sixteen free SMs in one GPC).  Asked once per kernel and device; returns the
// number of such clusters the device holds at a time (0: none, or the query failed).
template <auto kern>                                     // (one set of flags per kernel, not per kernel type)
int clusters_of_sixteen(int threads, int bytes) {
    static std::atomic<uint64_t> asked{0};
    static std::atomic<int> resident[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    const uint64_t bit = 1ull << dev;
    if (!(asked.load(std::memory_order_acquire) & bit)) {
        int n = 0;
        bool good = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
        if (good) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3(16, 1);
            q.blockDim = dim3(threads);
            q.dynamicSmemBytes = bytes;
            cudaLaunchAttribute a[1];
            a[0].id = cudaLaunchAttributeClusterDimension;
            a[0].val.clusterDim.x = 16; a[0].val.clusterDim.y = 1; a[0].val.clusterDim.z = 1;
            q.attrs = a;
            q.numAttrs = 1;
            good = cudaOccupancyMaxActiveClusters(&n, kern, &q) == cudaSuccess && n >= 1;
        }
        if (!good) { cudaGetLastError(); n = 0; }
        resident[dev].store(n, std::memory_order_release);
        asked.fetch_or(bit, std::memory_order_release);
    }
    return resident[dev].load(std::memory_order_acquire);
}

template <int D, int NT>
int launch_tc2_d(const Problem& p, cudaStream_t st, int key_split = 1, bool only_if_resident = false) {
    using LY = L2<D, NT>;
    CUtensorMap tmQ, tmK, tmV;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, D, BM) || !make_map(&tmK, p.K, BH, p.Nk, D, BN) ||
        !make_map(&tmV, p.V, BH, p.Nk, D, BN))
        return FLAT_ERR_CUDA;
    dim3 grid((p.Nq + NT * BM - 1) / (NT * BM), BH);
    if (p.block_mask) {
        if constexpr (NT == 1) {
            if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT, false, false, true>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
            fused_tc2_kernel<D, NT, false, false, true><<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(
                tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, p.scale * 1.4426950408889634f,
                p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status, nullptr, nullptr, p.lse,
                BiasArg{nullptr, 0, 0, 0, 0}, p.block_mask, p.bmask_sb, p.bmask_sh);
            return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
        } else {
            return FLAT_ERR_UNSUPPORTED;
        }
    }
    if (p.bias) {
        if constexpr (NT == 2 && D == 64) {
            // bf16 bias with 16-byte aligned rows: tiles staged through shared memory by TMA
            const BiasArg ba = bias_arg(p);
            CUtensorMap tmB;
            if (ba.vec && !ba.f32 && make_bias_map(&tmB, p)) {
                using LB = L2<D, NT, true>;
                if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT, false, 2>>(LB::SMEM_BYTES)) return FLAT_ERR_CUDA;
                fused_tc2_kernel<D, NT, false, 2><<<grid, LB::THREADS, LB::SMEM_BYTES, st>>>(
                    tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, p.scale * 1.4426950408889634f,
                    p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status, nullptr, nullptr, p.lse, ba, nullptr, 0, 0, tmB);
                return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
            }
        }
        if constexpr (NT == 2) {
            if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT, false, true>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
            fused_tc2_kernel<D, NT, false, true><<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(
                tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, p.scale * 1.4426950408889634f,
                p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status, nullptr, nullptr, p.lse, bias_arg(p));
            return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
        } else {
            return FLAT_ERR_UNSUPPORTED;
        }
    }
    if constexpr (NT == 1) {
        if (key_split == 2 || key_split == 4 || key_split == 8 || (key_split == 16 && D == 128)) {
            // the keys of every query tile over a cluster of 2, 4, 8 or 16 CTAs (consecutive along x)
            auto launch = [&](auto cs_tag) -> int {
                constexpr int CS = decltype(cs_tag)::value;
                constexpr int BYTES = LY::SMEM_BYTES + LY::merge_bytes(CS);
                if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT, false, false, false, CS>>(BYTES)) return FLAT_ERR_CUDA;
                if constexpr (CS > 8) {
                    // (the dispatcher only wants them when all clusters of the launch run at once: 8 clusters of sixteen
                    // one-per-SM CTAs took 80 us where clusters of eight take 41)
                    const int fit = clusters_of_sixteen<fused_tc2_kernel<D, NT, false, false, false, CS>>(LY::THREADS, BYTES);
                    if (fit < 1 || (only_if_resident && static_cast<int64_t>(grid.x) * grid.y > fit)) return FLAT_ERR_UNSUPPORTED;
                }
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(grid.x * CS, grid.y);
                cfg.blockDim = dim3(LY::THREADS);
                cfg.dynamicSmemBytes = BYTES;
                cfg.stream = st;
                cudaLaunchAttribute attr[2];
                attr[0].id = cudaLaunchAttributeClusterDimension;
                attr[0].val.clusterDim.x = CS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
                attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // (see the kernel's prologue)
                attr[1].val.programmaticStreamSerializationAllowed = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 2;
                const cudaError_t e = cudaLaunchKernelEx(
                    &cfg, fused_tc2_kernel<D, NT, false, false, false, CS>, tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H,
                    p.Nq, p.Nk, p.scale * 1.4426950408889634f, p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status,
                    static_cast<const int32_t*>(nullptr), static_cast<const int32_t*>(nullptr), p.lse,
                    BiasArg{nullptr, 0, 0, 0, 0}, static_cast<const uint8_t*>(nullptr), 0ll, 0ll, CUtensorMap{});
                return e == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
            };
            if constexpr (D == 128) {
                if (key_split == 16) return launch(std::integral_constant<int, 16>{});
            }
            return key_split == 2 ? launch(std::integral_constant<int, 2>{})
                   : key_split == 4 ? launch(std::integral_constant<int, 4>{}) : launch(std::integral_constant<int, 8>{});
        }
    }
    if (key_split != 1) return FLAT_ERR_UNSUPPORTED;
    auto kern = fused_tc2_kernel<D, NT>;
    if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
    if constexpr (NT == 1) {
        // short launches: the kernel may start while its predecessor in the stream drains (see its prologue)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(LY::THREADS);
        cfg.dynamicSmemBytes = LY::SMEM_BYTES;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t e = cudaLaunchKernelEx(
            &cfg, kern, tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, p.scale * 1.4426950408889634f,
            p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status, static_cast<const int32_t*>(nullptr),
            static_cast<const int32_t*>(nullptr), p.lse, BiasArg{nullptr, 0, 0, 0, 0}, static_cast<const uint8_t*>(nullptr), 0ll, 0ll,
            CUtensorMap{});
        return e == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
    }
    kern<<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq,
                                                    p.Nk, p.scale * 1.4426950408889634f, p.k_valid_len,
                                                    p.causal ? p.Nk - p.Nq : (1 << 30), p.status, nullptr, nullptr, p.lse,
                                                    BiasArg{nullptr, 0, 0, 0, 0}, nullptr, 0, 0, CUtensorMap{});
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

// Key halves (see the kernel's KH): d = 64, dense, one 128-row tile per CTA worked on by two warpgroups, optionally
// with the keys over a cluster on top.  One CTA per SM (all 512 TMEM columns).
int launch_tc2_kh(const Problem& p, cudaStream_t st, int key_split, bool only_if_resident) {
    constexpr int D = 64, NT = 2;
    CUtensorMap tmQ, tmK, tmV;
    const int BH = p.B * p.H;
    if (!make_map(&tmQ, p.Q, BH, p.Nq, D, BM) || !make_map(&tmK, p.K, BH, p.Nk, D, BN) ||
        !make_map(&tmV, p.V, BH, p.Nk, D, BN))
        return FLAT_ERR_CUDA;
    const dim3 grid((p.Nq + BM - 1) / BM, BH);
    auto launch = [&](auto cs_tag) -> int {
        constexpr int CS = decltype(cs_tag)::value;
        using LY = L2<D, NT, false, CS == 16 ? 2 : 1>;   // (the kernel's own choice of ring depths)
        constexpr int BYTES = LY::SMEM_BYTES + LY::merge_bytes(CS) + 128 * merge_vecs(D) * 16;
        static_assert(BYTES <= 232448, "shared memory of the two-warpgroup form");
        auto kern = fused_tc2_kernel<D, NT, false, 0, false, CS, true>;
        if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT, false, 0, false, CS, true>>(BYTES)) return FLAT_ERR_CUDA;
        if constexpr (CS > 8) {
            const int fit = clusters_of_sixteen<fused_tc2_kernel<D, NT, false, 0, false, CS, true>>(LY::THREADS, BYTES);
            if (fit < 1 || (only_if_resident && static_cast<int64_t>(grid.x) * grid.y > fit)) return FLAT_ERR_UNSUPPORTED;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid.x * CS, grid.y);
        cfg.blockDim = dim3(LY::THREADS);
        cfg.dynamicSmemBytes = BYTES;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // (see the kernel's prologue)
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = CS; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = CS > 1 ? 2 : 1;
        const cudaError_t e = cudaLaunchKernelEx(
            &cfg, kern, tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.O), p.H, p.Nq, p.Nk, p.scale * 1.4426950408889634f,
            p.k_valid_len, p.causal ? p.Nk - p.Nq : (1 << 30), p.status, static_cast<const int32_t*>(nullptr),
            static_cast<const int32_t*>(nullptr), p.lse, BiasArg{nullptr, 0, 0, 0, 0}, static_cast<const uint8_t*>(nullptr), 0ll, 0ll,
            CUtensorMap{});
        return e == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
    };
    return key_split == 1   ? launch(std::integral_constant<int, 1>{})
           : key_split == 2 ? launch(std::integral_constant<int, 2>{})
           : key_split == 4 ? launch(std::integral_constant<int, 4>{})
           : key_split == 8 ? launch(std::integral_constant<int, 8>{})
           : key_split == 16 ? launch(std::integral_constant<int, 16>{}) : FLAT_ERR_UNSUPPORTED;
}

}  // namespace


int launch_fused_tc2_varlen(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_q,
                            const int32_t* cu_k, int num_seqs, int H, int64_t total_q, int64_t total_k,
                            int max_seqlen_q, float scale, int causal, int32_t* status, cudaStream_t st) {
    constexpr int D = 128, NT = 2;
    using LY = L2<D, NT>;
    if (static_cast<int64_t>(num_seqs) * H > 65535) return FLAT_ERR_SHAPE;      // (grid y)
    CUtensorMap tmQ, tmK, tmV;
    if (!make_map_packed(&tmQ, Q, total_q, H, D, BM) || !make_map_packed(&tmK, K, total_k, H, D, BN) ||
        !make_map_packed(&tmV, V, total_k, H, D, BN))
        return FLAT_ERR_CUDA;
    if (!ensure_dynamic_smem<fused_tc2_kernel<D, NT, true>>(LY::SMEM_BYTES)) return FLAT_ERR_CUDA;
    dim3 grid((max_seqlen_q + NT * BM - 1) / (NT * BM), num_seqs * H);
    fused_tc2_kernel<D, NT, true><<<grid, LY::THREADS, LY::SMEM_BYTES, st>>>(
        tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(O), H, max_seqlen_q, 0, scale * 1.4426950408889634f, nullptr,
        causal ? 0 : (1 << 30), status, cu_q, cu_k);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

namespace {

// Self-test of the give-up path: one warp waits on a barrier that nothing will ever complete, with
// a limit of about a tenth of a second.  The wait must run out, record its code and let the kernel
// end normally (no trap, no hang), leaving the context usable.
__global__ void wait_timeout_selftest_kernel(int32_t* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; fence_mbar_init(); }
    __syncthreads();
    const bool ok = bounded_wait(&bar, 0, &abort_flag, status, 0x7e57, 200000000ll);
    if (ok && threadIdx.x == 0 && status) atomicExch(status, -1);   // would mean the wait "succeeded"
}

// Self-test of the polynomial exponential: y[i] = ex2_poly(x[i]).
__global__ void exp2_poly_selftest_kernel(const float* __restrict__ x, float* __restrict__ y, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) y[i] = ex2_poly(x[i]);
}

}  // namespace

int launch_exp2_poly_selftest(const float* x, float* y, int n, cudaStream_t st) {
    exp2_poly_selftest_kernel<<<(n + 255) / 256, 256, 0, st>>>(x, y, n);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

int launch_wait_timeout_selftest(int32_t* status, cudaStream_t st) {
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(status);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

int launch_fused_tc2(const Problem& p, cudaStream_t st) {
    if (p.dtype != FLAT_DTYPE_BF16) return FLAT_ERR_UNSUPPORTED;
    if (p.d == 64) return launch_tc2_d<64, 2>(p, st);
    if (p.d == 128) return launch_tc2_d<128, 2>(p, st);
    return FLAT_ERR_UNSUPPORTED;
}

int launch_fused_tc2_halves(const Problem& p, cudaStream_t st, int key_split, bool only_if_resident) {
    if (p.dtype != FLAT_DTYPE_BF16 || p.d != 64 || p.bias || p.block_mask) return FLAT_ERR_UNSUPPORTED;
    return launch_tc2_kh(p, st, key_split, only_if_resident);
}

// One 128-row tile per CTA, two CTAs per SM (d = 64 only: at d = 128 two CTAs do not fit in shared memory).
int launch_fused_tc2_single(const Problem& p, cudaStream_t st, int key_split, bool only_if_resident) {
    if (p.dtype != FLAT_DTYPE_BF16) return FLAT_ERR_UNSUPPORTED;
    if (key_split != 1 && (p.bias || p.block_mask)) return FLAT_ERR_UNSUPPORTED;
    if (p.d == 64) return launch_tc2_d<64, 1>(p, st, key_split);
    if (key_split == 16 && p.d != 128) return FLAT_ERR_UNSUPPORTED;      // (sixteen-CTA clusters: built for d = 128, one CTA per SM)
    if (p.d == 128 && (p.block_mask || key_split != 1)) return launch_tc2_d<128, 1>(p, st, key_split, only_if_resident);   // (one CTA per SM: the pruned path and the key split)
    return FLAT_ERR_UNSUPPORTED;
}

}  // namespace flat

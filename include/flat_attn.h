/*
 * flat_attn.h -- C ABI of the fused exact-attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes O = softmax(scale * Q K^T) V for multi-head attention
 * (paper Section 2, "Computation operators", steps 2-4: Logit, Softmax along
 * the key index, Attend) in two ways:
 *
 *   - fused (the paper's FLAT dataflow, Section 5 and 5.1): the outer loops over
 *     batch, head and query-row tile are shared by the Logit and Attend
 *     operators, the slice of the logit tensor produced by Logit is consumed by
 *     Softmax and Attend on chip, and only Q, K, V are read and O is written;
 *   - naive (the paper's baseline, Section 4.2 and Fig. 7(a)): operator by
 *     operator, with the [B,H,Nq,Nk] logit tensor L and weight tensor A written
 *     to and read back from device memory.
 *
 * Conventions for every entry point
 *   - Tensors are dense, row-major, innermost dimension contiguous:
 *       Q, O : [B, H, Nq, d]      K, V : [B, H, Nk, d]      L, A : [B, H, Nq, Nk]
 *   - Unless an argument says HOST, pointers are DEVICE pointers owned by the
 *     caller, 16-byte aligned.  The library allocates and frees no device memory
 *     and keeps no pointer after a call returns.  (What it needs beyond the caller's
 *     buffers lives in its own device image: a status word, the workspace of the
 *     even deal -- see flat_attn_last_schedule -- and that of flat_attn_naive_fwd_static.
 *     The even deal also records one event per launch, created once per device.)
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream); the library does not synchronise unless stated.
 *   - Return value: FLAT_OK or one of the error codes below.  On an argument
 *     error nothing is launched.  There is no CPU fallback: an unsupported
 *     request is an error.
 *   - Supported sizes: B, H, Nq, Nk >= 1; d in {16, 32, 64, 128} (tensor-core
 *     kernels need d in {64, 128} and bf16); B*H*Nq*Nk and all byte counts must
 *     fit in 63 bits; B*H <= 65535.
 *   - scale multiplies the logits before the softmax and must be finite.  The
 *     paper does not mention a scale (scale = 1 is its literal text); 1/sqrt(d)
 *     is the usual choice.
 *   - Key-padding mask (k_valid_len, optional): key j of batch b takes part iff
 *     j < k_valid_len[b], for all heads and query rows; values must lie in
 *     [0, Nk].  Masked K/V entries must be finite and are otherwise ignored.  A
 *     batch with k_valid_len[b] == 0 gets O = 0 (and A = 0).
 */
#ifndef FLAT_ATTN_H_
#define FLAT_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    FLAT_OK = 0,
    FLAT_ERR_NULL = 1,         /* a required pointer is NULL                                  */
    FLAT_ERR_SHAPE = 2,        /* a size is < 1, overflows, or k_valid_len is out of range     */
    FLAT_ERR_UNSUPPORTED = 3,  /* d, dtype or variant not supported by any kernel              */
    FLAT_ERR_ALIGN = 4,        /* a pointer is not 16-byte aligned                             */
    FLAT_ERR_WORKSPACE = 5,    /* caller-provided workspace too small                          */
    FLAT_ERR_CUDA = 6,         /* a CUDA runtime/driver call failed (launch, tensor map, copy) */
    FLAT_ERR_TIMEOUT = 7       /* a bounded device-side wait gave up (reported via `status`)   */
};

enum { FLAT_DTYPE_BF16 = 0, FLAT_DTYPE_F32 = 1 };

/* Kernel choice for the fused path. AUTO picks the tensor-core kernel when it applies. */
enum {
    FLAT_VARIANT_AUTO = 0,
    FLAT_VARIANT_SIMT = 1,     /* fp32 FFMA kernel, any supported d and dtype                  */
    FLAT_VARIANT_TC = 2,       /* tcgen05 + TMEM + TMA kernel, one 128-row tile per CTA:
                                  bf16, d in {64,128}                                          */
    FLAT_VARIANT_TC2 = 3,      /* same, two 128-row tiles per CTA ping-ponging on the tensor
                                  pipe (the default for problems that fill the GPU)            */
    FLAT_VARIANT_TC2_SINGLE = 4, /* the TC2 pipeline with one 128-row tile per CTA and two CTAs
                                  per SM: bf16, d = 64 only                                    */
    FLAT_VARIANT_TC3 = 5,      /* two tiles per CTA, the softmax of every row split over two
                                  threads (sixteen softmax warps), logit tiles computed three
                                  tile-steps ahead in rotating TMEM buffers: bf16, d = 64 only */
    FLAT_VARIANT_RGRAN = 6,    /* the paper's row-granularity dataflow taken literally: the whole
                                  row of logits of a 128-row tile stays on chip (TMEM), two-pass
                                  softmax over complete rows: bf16, d = 64, Nk <= 512 only      */
    FLAT_VARIANT_TF32 = 7,     /* fp32 tensors on the tensor cores: every operand split into a tf32
                                  head and an fp32 remainder, each contraction three tf32 products,
                                  running sums in fp32 registers: fp32, d = 64, no bias, no
                                  pruning map (what AUTO picks there)                            */
    FLAT_VARIANT_TC2_SPLIT2 = 8, /* TC2_SINGLE with the keys of every query tile split over a cluster
                                  of two CTAs, whose partial softmaxes are merged through
                                  distributed shared memory: bf16, d in {64,128}, no bias, no pruning map;
                                  what AUTO picks at d = 128 for launches that would leave most
                                  SMs empty (at d = 64 it takes the HALVES forms below)          */
    FLAT_VARIANT_TC2_SPLIT4 = 9, /* the same over a cluster of four CTAs                           */
    FLAT_VARIANT_TC2_SPLIT8 = 10, /* the same over a cluster of eight CTAs                          */
    FLAT_VARIANT_TC2_HALVES = 11, /* one 128-row tile per CTA worked on by two softmax warpgroups, which take the
                                  even and the odd key tiles and merge their partial softmaxes through shared
                                  memory at the end (half the chain of key steps that a short launch waits for):
                                  bf16, d = 64, no bias, no pruning map; one CTA per SM; what AUTO picks,
                                  with the largest cluster that fits, while every CTA gets an SM of its own */
    FLAT_VARIANT_TC2_HALVES_SPLIT2 = 12, /* the same with the keys also split over a cluster of two CTAs     */
    FLAT_VARIANT_TC2_HALVES_SPLIT4 = 13, /* ... of four CTAs                                             */
    FLAT_VARIANT_TC2_HALVES_SPLIT8 = 14, /* ... of eight CTAs                                            */
    FLAT_VARIANT_TC2_SPLIT16 = 15, /* TC2_SPLIT2 over a cluster of sixteen CTAs (more than the portable cluster size:
                                  taken only where the device can hold such a cluster): bf16, d = 128       */
    FLAT_VARIANT_TC2_HALVES_SPLIT16 = 16 /* TC2_HALVES over a cluster of sixteen CTAs: bf16, d = 64               */
};

typedef struct flat_attn_params {
    const void* Q;             /* [B,H,Nq,d]                                                   */
    const void* K;             /* [B,H,Nk,d]                                                   */
    const void* V;             /* [B,H,Nk,d]                                                   */
    void* O;                   /* [B,H,Nq,d], same dtype as the inputs                         */
    int B, H, Nq, Nk, d;
    float scale;
    int dtype;                 /* FLAT_DTYPE_BF16 or FLAT_DTYPE_F32 (storage of Q,K,V,O);
                                  accumulation is always fp32                                 */
    const int32_t* k_valid_len;/* device, [B], or NULL = all keys valid                        */
    int32_t* status;           /* optional device word; a kernel that gives up on a bounded
                                  wait stores a non-zero code here (never traps or hangs).
                                  NULL: the code goes to the library's own device word instead,
                                  see flat_attn_last_device_error                              */
    int variant;               /* FLAT_VARIANT_*                                               */
    int causal;                /* 0, or 1 = causal mask: query i takes part with key j iff
                                  j <= i + (Nk - Nq) (the last query sees every key), intersected
                                  with k_valid_len.  The paper names masking only in passing
                                  (Section 2, footnote); its decoder workloads need it.  The
                                  unfused baseline honours it too (A is 0 beyond the limit).    */
    float* lse;                /* optional device output [B,H,Nq] fp32 (4-byte aligned), fused
                                  path only: lse[b,h,i] = log sum_j exp(scale * q_i . k_j) over the
                                  keys that row i sees (natural logarithm; -inf for a row without
                                  any).  It is what flat_attn_bwd needs from the forward pass.
                                  Written by the SIMT, TC2, TC2_SINGLE and TC3 kernels (AUTO picks
                                  among these when it is set); FLAT_ERR_UNSUPPORTED for the others.
                                  The paper has no counterpart (it stops at inference).           */
    const void* bias;          /* optional device tensor added to the SCALED logits before the
                                  softmax (it is not multiplied by `scale`): the relative-position
                                  terms of the paper's T5 / TrXL workloads (Section 6.1), which the
                                  paper itself does not model.  Element (b,h,i,j) is read at
                                  b * bias_stride_b + h * bias_stride_h + i * Nk + j (rows dense);
                                  a stride of 0 repeats the values for every batch / head.  -inf
                                  switches a (query, key) pair off; a row with every pair off gives
                                  O = 0.  Aligned to its element size (16-byte alignment of the
                                  base, the strides and Nk lets the kernel use vector loads).
                                  Fused path only; run by the SIMT and TC2 kernels (AUTO picks TC2
                                  for bf16 with d in {64,128}); FLAT_ERR_UNSUPPORTED for the other
                                  variants.  NULL = none.                                         */
    int bias_dtype;            /* FLAT_DTYPE_BF16 or FLAT_DTYPE_F32 (storage of `bias`)            */
    long long bias_stride_b, bias_stride_h;   /* in elements, >= 0                               */
    const uint8_t* block_mask; /* optional device byte map for PRUNED (sparse) Logit-Attend (paper
                                  Section 8.2 studies randomly pruned attention): one byte per
                                  128 x 128 block of the logit matrix, [B or 1, H or 1,
                                  ceil(Nq/128), ceil(Nk/128)], read at b * block_mask_stride_b +
                                  h * block_mask_stride_h + tq * ceil(Nk/128) + tk.  A block whose
                                  byte is 0 takes no part: its key tile is neither loaded nor
                                  multiplied for that query tile (the work and the K/V traffic
                                  shrink with the density); a query row whose every block is pruned
                                  gives O = 0.  Combines with k_valid_len, causal and lse, not with
                                  bias.  bf16, d in {64, 128}, Nk <= 131072; run by the one-tile
                                  tensor-core kernel (AUTO picks it); FLAT_ERR_UNSUPPORTED otherwise.
                                  NULL = dense.                                                   */
    long long block_mask_stride_b, block_mask_stride_h;   /* in bytes (= elements), >= 0         */
} flat_attn_params_t;

/*
 * Fused attention, bf16 in / bf16 out, fp32 accumulation, no mask.
 * Operation: paper Section 5 (fused Logit-Softmax-Attend loop nest, row granularity,
 * Section 5.2) applied to the operators of Section 2 steps 2-4.
 * Equivalent to flat_attn_fwd_ex with dtype = BF16, k_valid_len = NULL, variant = AUTO.
 */
int flat_attn_fwd(const void* Q, const void* K, const void* V, void* O,
                  int B, int H, int Nq, int Nk, int d, float scale, void* stream);

/* Fused attention with dtype choice, optional key-padding mask, optional causal mask and
 * kernel choice (same operation as flat_attn_fwd; a masked key takes no part in the softmax of
 * the row, a row without any key gives O = 0).  `p` is a HOST pointer, read before the call
 * returns.  FLAT_VARIANT_TC does not implement the causal mask (FLAT_ERR_UNSUPPORTED). */
int flat_attn_fwd_ex(const flat_attn_params_t* p, void* stream);

/*
 * The paper's unfused baseline (Section 4.2; Fig. 7(a)): three kernels,
 *   L = scale * Q K^T   written to device memory as fp32 [B,H,Nq,Nk],
 *   A = softmax_row(L)  written as bf16 (dtype BF16) or fp32 (dtype F32) [B,H,Nq,Nk],
 *   O = A V.
 * L and A are caller-allocated device buffers; their contents after the call are
 * the logits (all columns, masked ones included, unmasked values) and the weights
 * (masked columns 0).  The row softmax runs one thread block per row of L, so B*H*Nq must not
 * exceed 2^31 - 1 (FLAT_ERR_SHAPE, nothing launched).
 */
int flat_attn_naive_fwd(const void* Q, const void* K, const void* V, void* O, void* L, void* A,
                        int B, int H, int Nq, int Nk, int d, float scale, void* stream);
int flat_attn_naive_fwd_ex(const flat_attn_params_t* p, void* L, void* A, void* stream);

/*
 * Backward pass of the fused attention: gradients dQ, dK, dV of a scalar loss, given dO = dLoss/dO.
 * The paper describes the forward operators only; this is the chain rule on its Section 2 steps 2-4,
 * run with the idea of its Section 5: the [B,H,Nq,Nk] intermediates (the weights, their gradient and
 * the logit gradient) are rebuilt tile by tile on chip from Q, K, V and the forward's `lse`, and never
 * reach device memory.  With S = scale Q K^T, P = exp(S - lse) and delta_i = sum_t dO[i,t] O[i,t]:
 *     dV = P^T dO      dP = dO V^T      dS = P o (dP - delta)      dQ = scale dS K      dK = scale dS^T Q
 * Masks as in the forward (k_valid_len, causal): masked (query, key) pairs carry no gradient, masked
 * keys get dK = dV = 0, a query row without any visible key gets dQ = 0.
 *   Q, O, dO, dQ : [B,H,Nq,d] bf16      K, V, dK, dV : [B,H,Nk,d] bf16      (16-byte aligned)
 *   lse          : [B,H,Nq] fp32, as written by flat_attn_fwd_ex (params.lse) for the same inputs
 *   delta        : [B,H,Nq] fp32 scratch owned by the caller (4-byte aligned); overwritten
 * Two kernels are enqueued on `stream` (dQ and delta; then dK and dV), no atomics, results are
 * bit-reproducible.  bf16 only, d in {64, 128} (FLAT_ERR_UNSUPPORTED otherwise: no fallback); other
 * argument rules and error codes as for flat_attn_fwd_ex; nothing is launched on an argument error.
 * `p` is a HOST pointer, read before the call returns.
 */
typedef struct flat_attn_bwd_params {
    const void *Q, *K, *V, *O, *dO;
    const float* lse;
    void *dQ, *dK, *dV;
    float* delta;
    int B, H, Nq, Nk, d;
    float scale;
    const int32_t* k_valid_len;/* device, [B], or NULL                                          */
    int32_t* status;           /* optional device word, as in flat_attn_params_t                */
    int causal;                /* 0 / 1, as in flat_attn_params_t                                */
} flat_attn_bwd_params_t;
int flat_attn_bwd_ex(const flat_attn_bwd_params_t* p, void* stream);
int flat_attn_bwd(const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* lse,
                  void* dQ, void* dK, void* dV, float* delta,
                  int B, int H, int Nq, int Nk, int d, float scale, void* stream);

/*
 * Fused attention over a PACKED batch of sequences of different lengths (no padding): the same
 * operation as flat_attn_fwd_ex (paper Section 5 applied to Section 2 steps 2-4), sequence by
 * sequence.  Q, O are [total_q, H, d] and K, V [total_k, H, d], bf16, row-major (d contiguous, then
 * the head, then the token); sequence s owns the query tokens cu_seqlens_q[s] .. cu_seqlens_q[s+1]-1
 * and the key tokens cu_seqlens_k[s] .. cu_seqlens_k[s+1]-1.  cu_seqlens_q / _k are DEVICE arrays
 * of num_seqs + 1 non-decreasing int32 offsets, the first 0, the last total_q / total_k; they are
 * read by the kernel, not by the host.  max_seqlen_q >= the longest query sequence (it sizes the
 * grid; a larger value only adds empty work items).  causal = 1: query i of a sequence sees key j
 * of the same sequence iff j <= i + (its key count - its query count).  A query row without any
 * visible key gives O = 0.  The paper works on dense [B,H,N,d] batches; packing is this library's
 * way of running its workloads' real length mixes without padding.
 * Needs d in {64, 128} (FLAT_ERR_UNSUPPORTED otherwise: no fallback) and, at d = 128,
 * num_seqs * H <= 65535.  All pointers are device pointers, 16-byte aligned (the offset arrays
 * 4-byte); `status` as in flat_attn_params_t.
 */
int flat_attn_varlen_fwd(const void* Q, const void* K, const void* V, void* O,
                         const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k,
                         int num_seqs, int H, int d, long long total_q, long long total_k,
                         int max_seqlen_q, float scale, int causal, int32_t* status, void* stream);

/*
 * The activation-weight operators of an attention layer (paper Section 2, "Computation
 * operators": step 1, the Query / Key / Value projections of the input; step 5, the Output
 * projection of the concatenated heads).  bf16 operands, fp32 accumulation, bf16 results; the
 * paper names no bias and none is applied.  All pointers are DEVICE pointers owned by the
 * caller, 16-byte aligned; `status` is an optional device word as in flat_attn_params_t.
 *
 * flat_qkv_proj_fwd:  X [B,N,Dm] row-major (Dm contiguous); Wqkv [3*H*d, Dm] row-major, its
 *   rows being the H*d output features of Query, then Key, then Value, head by head;
 *   Q, K, V [B,H,N,d]:   Q[b,h,n,c] = sum_k X[b,n,k] * Wqkv[h*d + c, k]   (K, V: rows offset by
 *   H*d and 2*H*d).  One contraction; the results are written head-major, the layout the fused
 *   attention reads.  Needs d in {64,128}, H*d a multiple of 256, Dm a multiple of 64.
 * flat_out_proj_fwd:  O [B,H,N,d]; Wo [Dm, H*d] row-major; Y [B,N,Dm]:
 *   Y[b,n,j] = sum_{h,c} O[b,h,n,c] * Wo[j, h*d + c].  Needs d in {64,128}, N a multiple of
 *   128, Dm a multiple of 256.
 * flat_attn_layer_fwd:  steps 1-5 of Section 2 for self-attention: the Q/K/V projection, the
 *   fused Logit-softmax-Attend (flat_attn_fwd_ex with dtype BF16, no key-padding mask, `causal`
 *   as given) and the Output projection, enqueued on `stream` in this order.  Q, K, V, O are
 *   caller-owned device buffers of B*H*N*d bf16 elements each that hold the intermediates (the
 *   library allocates nothing); their contents after the call are those intermediates.
 *   Needs every condition of the two projections.
 * Errors: FLAT_ERR_NULL / SHAPE / UNSUPPORTED / ALIGN as above; nothing is launched on an
 * argument error.
 */
int flat_qkv_proj_fwd(const void* X, const void* Wqkv, void* Q, void* K, void* V,
                      int B, int N, int H, int d, int Dm, int32_t* status, void* stream);
int flat_out_proj_fwd(const void* O, const void* Wo, void* Y,
                      int B, int N, int H, int d, int Dm, int32_t* status, void* stream);
int flat_attn_layer_fwd(const void* X, const void* Wqkv, const void* Wo, void* Y,
                        void* Q, void* K, void* V, void* O,
                        int B, int N, int H, int d, int Dm, float scale, int causal,
                        int32_t* status, void* stream);

/*
 * A fully connected operator of the attention block (the layers that follow the attention and
 * normalisation layers of a block, paper Section 2; FF1 / FF2 of Table 2):  Y [M, Nout] = X [M, K] * W[Nout, K]^T, all row-major bf16, fp32 accumulation, no
 * bias and no activation (the paper names none).  The same kernel as the projections.  Needs K a
 * multiple of 64 and Nout a multiple of 256.  DEVICE pointers, 16-byte aligned; errors as above.
 */
int flat_fc_fwd(const void* X, const void* W, void* Y, int M, int K, int Nout, int32_t* status, void* stream);

/*
 * The normalisation layer of an attention block (paper Section 2 lists it between the attention layer
 * and the fully connected layers and says no more).  Reading taken: layer normalisation of every token
 * over its D features, after the residual add:
 *     z = X + R  (R may be NULL: z = X),    Y = gamma * (z - mean(z)) / sqrt(var(z) + eps) + beta
 * with the biased variance (divided by D).  X, R, Y: [M, D] row-major bf16; gamma, beta: [D] bf16;
 * statistics in fp32.  Y may alias X or R.  Needs D a multiple of 8 and at most 8192
 * (FLAT_ERR_UNSUPPORTED otherwise), eps >= 0; DEVICE pointers, 16-byte aligned.  One kernel, bound by
 * device-memory bandwidth (each element read once, written once).
 */
int flat_layernorm_fwd(const void* X, const void* R, const void* gamma, const void* beta, void* Y,
                       long long M, int D, float eps, void* stream);

/*
 * End-to-end convenience call with HOST tensors: copies Q, K, V (and k_valid_len if
 * non-NULL) from host memory into `workspace`, runs the fused kernel, copies O back
 * to `O_host`, and returns without synchronising (use pinned host memory for true
 * asynchrony; the caller synchronises `stream` before reading O).  The work is cut
 * into up to 8 independent slices (whole batches, or groups of heads when B == 1)
 * that run on two internal side streams forked from and joined back into `stream`,
 * so that the transfer of one slice overlaps the kernel and the read-back of its
 * neighbours; to the caller it behaves like work enqueued on `stream`.  The side
 * streams and events are created once per device and host thread and never freed
 * (no device memory is allocated).
 * p->Q, p->K, p->V, p->O and p->k_valid_len are HOST pointers here; p->status and
 * p->lse are still device pointers or NULL.  `workspace` is a caller-owned DEVICE buffer of at
 * least flat_attn_host_workspace_bytes(...) bytes, 256-byte aligned.
 * The operation is that of flat_attn_fwd_ex; the paper has no counterpart for the copies.
 */
int flat_attn_fwd_host(const flat_attn_params_t* p, void* workspace, size_t workspace_bytes, void* stream);
size_t flat_attn_host_workspace_bytes(int B, int H, int Nq, int Nk, int d, int dtype);

/*
 * The unfused baseline for callers that cannot allocate device memory.
 *
 * (The paper has no counterpart for this entry point; the arithmetic is that of
 * flat_attn_naive_fwd: bf16 in and out, no mask.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin handed a
 * fixed memory budget by its host application, a real-time or safety-reviewed loop
 * that must not enter the driver's allocator (it can block, fail, or fragment the
 * budget), a process whose device memory was carved up at start-up.  Such a caller
 * can own Q, K, V and O but has nowhere to put the [B,H,Nq,Nk] logit and weight
 * tensors that the baseline materialises.  Here they live in a device array that is
 * part of the library image itself: fp32 logits followed by bf16 weights,
 * 6 * FLAT_STATIC_MAX_ELEMS bytes (24 MiB), resident on every GPU that loads the
 * library until the process exits.  The call path performs no cudaMalloc, cudaFree
 * or other allocating call.
 *
 *   - Limit: B*H*Nq*Nk <= FLAT_STATIC_MAX_ELEMS, otherwise FLAT_ERR_WORKSPACE is
 *     returned before anything touches the device.  Other argument rules and error
 *     codes are those of flat_attn_naive_fwd; Q, K, V, O stay caller-owned.
 *   - Arguments are checked first (size gate, then pointers, d, alignment), before the
 *     device is looked at.  The first valid call on each device then looks up the array's
 *     device address (with that device current, which is the caller's job as for every
 *     entry point); this is also the latest moment at which the CUDA runtime makes the
 *     array resident on that device, so it is the one call that can fail for lack of
 *     device memory (FLAT_ERR_CUDA).  Make one small warm-up call per device at start-up,
 *     outside any stream capture; later calls only enqueue the three kernels.
 *   - All calls on a device share the one array, and it keeps whatever the last call
 *     left in it.  The three kernels overwrite every element they later read, so
 *     nothing has to be cleared, but two calls whose kernels overlap on the GPU
 *     (different streams, different host threads) race on it: serialise them.
 */
#define FLAT_STATIC_MAX_ELEMS (4 * 1024 * 1024)
int flat_attn_naive_fwd_static(const void* Q, const void* K, const void* V, void* O,
                               int B, int H, int Nq, int Nk, int d, float scale, void* stream);

/*
 * Self-test of the device-side give-up path (the paper has no counterpart).  Every wait inside the
 * tensor-core kernels is bounded; when one runs out, the kernel stores a non-zero code in the
 * caller's `status` word and returns normally.  This call launches a one-warp kernel that waits,
 * for about 0.1 s, on a barrier nothing completes, and must leave FLAT_SELFTEST_TIMEOUT_CODE in
 * *status (a device int32, zeroed by the caller) with the context still usable afterwards.  With
 * status == NULL the code goes where every kernel's goes in that case: to the library's own word
 * (flat_attn_last_device_error).
 */
#define FLAT_SELFTEST_TIMEOUT_CODE 0x7e57
int flat_attn_selftest_wait_timeout(int32_t* status, void* stream);

/*
 * Self-test of the polynomial 2^x that the fused kernel uses for a quarter of its exponentials
 * (the paper has no counterpart): y[i] = 2^clamp(x[i], -126, 126) evaluated by that routine, for
 * n device floats.  Relative error <= 1e-4 inside the clamp range.
 */
int flat_attn_selftest_exp2_poly(const float* x, float* y, int n, void* stream);

/* Number of kernels the most recent successful call on this thread launched. */
int flat_attn_last_launch_count(void);

/* The FLAT_VARIANT_* that the most recent fused call on this host thread ran (what
 * FLAT_VARIANT_AUTO resolved to for that problem on the current device); 0 before any call. */
int flat_attn_last_variant(void);

/*
 * How the most recent FLAT_VARIANT_TC3 launch on this host thread handed the work items (batch, head, slab of
 * 256 query rows) to the SMs -- the tile order of the paper's Section 5.1 / 5.3: FLAT_SCHEDULE_ITEMS one CTA per
 * item, FLAT_SCHEDULE_PERSISTENT one CTA per SM walking a fixed share of the items, FLAT_SCHEDULE_EVEN_DEAL one
 * CTA per SM taking an equal share of the key steps of all items, items cut where a share ends and their
 * partial softmaxes merged through the library's own device workspace (chosen for few items of unequal
 * length -- key-padding masks -- or a last round that would stay mostly empty; not under the causal mask, not
 * with the lse output, not during stream capture, not while a launch from another stream may still use the
 * workspace).  0 before any such launch.
 */
#define FLAT_SCHEDULE_ITEMS 1
#define FLAT_SCHEDULE_PERSISTENT 2
#define FLAT_SCHEDULE_EVEN_DEAL 3
int flat_attn_last_schedule(void);

/*
 * Device-side give-up codes when the caller passed no `status` word (the paper has no
 * counterpart).  Every wait inside the tensor-core kernels is bounded (about a second of SM
 * clock, which also runs while a context is time-sliced out on a GPU shared with other
 * processes); a kernel whose wait runs out stores a code and returns, leaving O partly written,
 * after the host call has long returned FLAT_OK.  With status == NULL that code goes to one
 * sticky word per device inside the library.  flat_attn_last_device_error copies the word of
 * the current device to *code (HOST pointer; 0 = no kernel has given up since the last clear).
 * It is a blocking copy: synchronise the streams whose work you ask about first.
 * flat_attn_clear_device_error zeroes the word.  The first fused call on a device looks the
 * word's address up; make it outside any stream capture.
 */
int flat_attn_last_device_error(int32_t* code);
int flat_attn_clear_device_error(void);

const char* flat_attn_status_string(int code);
int flat_attn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FLAT_ATTN_H_ */

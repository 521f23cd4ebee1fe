// CPU oracle for exact multi-head attention, O = softmax(scale * Q K^T) V.
//
// TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA path is
// checked against; it is deliberately plain (double precision, one query row
// at a time, no blocking, no fusion, no vector intrinsics) and shares no code
// with the CUDA library.  Only the tests, the smoke check and the benchmark's
// CPU-baseline leg may call it.
//
// What it computes, in the paper's notation (Section 2, "Computation
// operators", steps 2-4; Q, K, V are [B, H, N, d] with d = D / H):
//   step 2, Logit  L[b,h,i,j] = sum_t Q[b,h,i,t] * K[b,h,j,t]   (a d-dim dot product)
//   step 3, Softmax over each row of logits, i.e. along the key index j
//           (the softmax reduces over the key index, Section 5.2)
//   step 4, Attend O[b,h,i,t] = sum_j A[b,h,i,j] * V[b,h,j,t]
// The fused dataflow (Section 5) claims the same function as the unfused
// chain, so the oracle is the definition written out.
//
// Readings where the paper is silent:
//   * scale multiplies the logit before the softmax (scale = 1 is the paper's text);
//     it arrives as a float and is widened to double, the value the GPU also gets.
//   * softmax subtracts the row maximum first (same function, no overflow).
//   * key-padding mask: key j of batch b takes part iff j < valid_len[b]; masked
//     keys are left out before the maximum.  A row with no valid key gives O = 0.
//   * Nq may differ from Nk (cross attention): softmax still runs along keys.
//   * additive bias (the relative-position terms of the paper's T5 / TrXL workloads, Section 6.1;
//     the paper does not model them): a tensor [B or 1, H or 1, Nq, Nk] added to the SCALED logit
//     before the maximum; -inf switches a pair off, a row with every pair off gives O = 0.
//   * pruned (sparse) Logit-Attend (Section 8.2 studies randomly pruned attention): a byte map over
//     tile x tile blocks of the logit matrix; a pruned block's pairs take no part (their logits count
//     as -inf), a row whose every block is pruned gives O = 0.
//   * causal mask (decoder workloads; the paper does not spell masks out): query i takes
//     part with key j iff j <= i + (Nk - Nq), i.e. the last query sees every key and each
//     earlier query one key fewer; combined with the key-padding mask by intersection.
//
// Parity pins (tests/test_oracle_pins.py): closed-form worked example, row sums,
// Q = 0 -> mean of V, identical keys -> uniform weights, key permutation, key
// shift, constant V / linearity, one-hot limit, split-merge identity, mask
// equivalence, brute force in long double on tiny shapes.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

inline double widen_bf16(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

struct Problem {
    const void* Q; const void* K; const void* V;
    int dtype;                       // 0: bf16 bit patterns (uint16), 1: float32
    int64_t B, H, Nq, Nk, d;
    double scale;
    const int32_t* valid_len;        // [B] or null
    int causal;                      // 0 / 1
    const int64_t* rows;             // flat row ids (b*H + h)*Nq + i, or null = all rows
    int64_t nrows;
    double* O;                       // [nrows, d]
    double* L;                       // [nrows, Nk] scaled logits, or null
    double* A;                       // [nrows, Nk] softmax weights, or null
    double* LSE;                     // [nrows] log of the row's sum of exponentials of the scaled logits, or null
    const void* bias;                // additive term of the logits, or null: element (b,h,i,j) at
    int bias_dtype;                  //   b * bias_sb + h * bias_sh + i * Nk + j  (0: bf16 bits, 1: float32);
    int64_t bias_sb, bias_sh;        //   a stride of 0 repeats the same values for every batch / head
    const uint8_t* bmask;            // pruned attention, or null: the pair (i, j) takes part iff byte
    int64_t bmask_sb, bmask_sh;      //   b * bmask_sb + h * bmask_sh + (i / tile) * ceil(Nk / tile) + j / tile is non-zero
    int64_t bmask_tile;              //   (tile x tile blocks of the logit matrix; strides of 0 repeat)
};

inline double elem(const void* base, int dtype, int64_t idx) {
    if (dtype == 0) return widen_bf16(static_cast<const uint16_t*>(base)[idx]);
    return static_cast<double>(static_cast<const float*>(base)[idx]);
}

// One query row: steps 2, 3, 4 in that order.
void attend_row(const Problem& p, int64_t r, std::vector<double>& s) {
    const int64_t row = p.rows ? p.rows[r] : r;
    const int64_t i = row % p.Nq;
    const int64_t bh = row / p.Nq;
    const int64_t b = bh / p.H;
    int64_t n = p.valid_len ? p.valid_len[b] : p.Nk;
    if (p.causal) {                  // keys 0 .. i + (Nk - Nq) only
        const int64_t lim = i + 1 + (p.Nk - p.Nq);
        if (lim < n) n = lim;
        if (n < 0) n = 0;
    }
    const int64_t qoff = (bh * p.Nq + i) * p.d;
    const int64_t koff = bh * p.Nk * p.d;
    double* o = p.O + r * p.d;
    double* lrow = p.L ? p.L + r * p.Nk : nullptr;
    double* arow = p.A ? p.A + r * p.Nk : nullptr;

    // Step 2: scaled logits of this query against every valid key.
    for (int64_t j = 0; j < n; ++j) {
        double acc = 0.0;
        for (int64_t t = 0; t < p.d; ++t)
            acc += elem(p.Q, p.dtype, qoff + t) * elem(p.K, p.dtype, koff + j * p.d + t);
        s[j] = p.scale * acc;
        // The bias joins the SCALED logit (it is not multiplied by scale) and takes part in the
        // maximum and the softmax like any logit; -inf switches the pair off.
        if (p.bias) s[j] += elem(p.bias, p.bias_dtype, b * p.bias_sb + (bh % p.H) * p.bias_sh + i * p.Nk + j);
        // A pruned block takes no part: its logits count as -inf.
        if (p.bmask) {
            const int64_t tk = (p.Nk + p.bmask_tile - 1) / p.bmask_tile;
            if (!p.bmask[b * p.bmask_sb + (bh % p.H) * p.bmask_sh + (i / p.bmask_tile) * tk + j / p.bmask_tile]) s[j] = -INFINITY;
        }
    }
    if (lrow) {
        for (int64_t j = 0; j < p.Nk; ++j) lrow[j] = (j < n) ? s[j] : -INFINITY;
    }

    for (int64_t t = 0; t < p.d; ++t) o[t] = 0.0;
    if (arow) for (int64_t j = 0; j < p.Nk; ++j) arow[j] = 0.0;
    if (p.LSE) p.LSE[r] = -INFINITY; // (the empty sum)
    if (n <= 0) return;              // no valid key: O = 0 by convention

    // Step 3: softmax along the key index.
    double m = s[0];
    for (int64_t j = 1; j < n; ++j) if (s[j] > m) m = s[j];
    if (m == -INFINITY) return;      // every pair switched off by the bias: as for a row without keys
    double l = 0.0;
    for (int64_t j = 0; j < n; ++j) { s[j] = std::exp(s[j] - m); l += s[j]; }
    if (p.LSE) p.LSE[r] = m + std::log(l);
    for (int64_t j = 0; j < n; ++j) s[j] /= l;
    if (arow) for (int64_t j = 0; j < n; ++j) arow[j] = s[j];

    // Step 4: weighted sum of the value vectors.
    for (int64_t j = 0; j < n; ++j) {
        const double a = s[j];
        for (int64_t t = 0; t < p.d; ++t)
            o[t] += a * elem(p.V, p.dtype, koff + j * p.d + t);
    }
}

void worker(const Problem* p, int64_t lo, int64_t hi) {
    std::vector<double> s(static_cast<size_t>(p->Nk > 0 ? p->Nk : 1));
    for (int64_t r = lo; r < hi; ++r) attend_row(*p, r, s);
}

}  // namespace

extern "C" {

// Returns 0 on success, 1 on a bad argument.  `nthreads` <= 0 means "all hardware
// threads"; the count actually used is written to *threads_used if non-null.
int oracle_attn_rows_sparse(const void* Q, const void* K, const void* V, int dtype,
                            int64_t B, int64_t H, int64_t Nq, int64_t Nk, int64_t d, float scale,
                            const int32_t* valid_len, int causal, const int64_t* rows, int64_t nrows,
                            double* O, double* L, double* A, double* LSE,
                            const void* bias, int bias_dtype, int64_t bias_sb, int64_t bias_sh,
                            const uint8_t* bmask, int64_t bmask_sb, int64_t bmask_sh, int64_t bmask_tile,
                            int nthreads, int* threads_used) {
    if (!Q || !K || !V || !O) return 1;
    if (B < 1 || H < 1 || Nq < 1 || Nk < 1 || d < 1) return 1;
    if (dtype != 0 && dtype != 1) return 1;
    if (bias && ((bias_dtype != 0 && bias_dtype != 1) || bias_sb < 0 || bias_sh < 0)) return 1;
    if (bmask && (bmask_tile < 1 || bmask_sb < 0 || bmask_sh < 0)) return 1;
    const int64_t total = B * H * Nq;
    if (!rows) nrows = total;
    if (nrows < 0) return 1;
    if (rows) for (int64_t r = 0; r < nrows; ++r) if (rows[r] < 0 || rows[r] >= total) return 1;
    if (valid_len) for (int64_t b = 0; b < B; ++b) if (valid_len[b] < 0 || valid_len[b] > Nk) return 1;

    Problem p{Q, K, V, dtype, B, H, Nq, Nk, d, static_cast<double>(scale), valid_len, causal ? 1 : 0, rows, nrows, O, L, A, LSE,
              bias, bias_dtype, bias_sb, bias_sh, bmask, bmask_sb, bmask_sh, bmask_tile};
    int nt = nthreads > 0 ? nthreads : static_cast<int>(std::thread::hardware_concurrency());
    if (nt < 1) nt = 1;
    if (nt > nrows) nt = nrows > 0 ? static_cast<int>(nrows) : 1;
    if (threads_used) *threads_used = nt;
    if (nrows == 0) return 0;
    std::vector<std::thread> pool;
    const int64_t per = (nrows + nt - 1) / nt;
    for (int w = 0; w < nt; ++w) {
        const int64_t lo = w * per, hi = (lo + per < nrows) ? lo + per : nrows;
        if (lo >= hi) break;
        pool.emplace_back(worker, &p, lo, hi);
    }
    for (auto& th : pool) th.join();
    return 0;
}

int oracle_attn_rows_bias(const void* Q, const void* K, const void* V, int dtype,
                          int64_t B, int64_t H, int64_t Nq, int64_t Nk, int64_t d, float scale,
                          const int32_t* valid_len, int causal, const int64_t* rows, int64_t nrows,
                          double* O, double* L, double* A, double* LSE,
                          const void* bias, int bias_dtype, int64_t bias_sb, int64_t bias_sh,
                          int nthreads, int* threads_used) {
    return oracle_attn_rows_sparse(Q, K, V, dtype, B, H, Nq, Nk, d, scale, valid_len, causal, rows, nrows, O, L, A, LSE,
                                   bias, bias_dtype, bias_sb, bias_sh, nullptr, 0, 0, 1, nthreads, threads_used);
}

int oracle_attn_rows_lse(const void* Q, const void* K, const void* V, int dtype,
                         int64_t B, int64_t H, int64_t Nq, int64_t Nk, int64_t d, float scale,
                         const int32_t* valid_len, int causal, const int64_t* rows, int64_t nrows,
                         double* O, double* L, double* A, double* LSE, int nthreads, int* threads_used) {
    return oracle_attn_rows_bias(Q, K, V, dtype, B, H, Nq, Nk, d, scale, valid_len, causal, rows, nrows, O, L, A, LSE,
                                 nullptr, 0, 0, 0, nthreads, threads_used);
}

int oracle_attn_rows(const void* Q, const void* K, const void* V, int dtype,
                     int64_t B, int64_t H, int64_t Nq, int64_t Nk, int64_t d, float scale,
                     const int32_t* valid_len, int causal, const int64_t* rows, int64_t nrows,
                     double* O, double* L, double* A, int nthreads, int* threads_used) {
    return oracle_attn_rows_lse(Q, K, V, dtype, B, H, Nq, Nk, d, scale, valid_len, causal, rows, nrows, O, L, A,
                                nullptr, nthreads, threads_used);
}

int oracle_hardware_threads(void) {
    int n = static_cast<int>(std::thread::hardware_concurrency());
    return n < 1 ? 1 : n;
}

}  // extern "C"

// CPU oracle for the gradient of exact multi-head attention.
//
// TEST INFRASTRUCTURE ONLY (see oracle_attn.cpp): plain double precision, one query row at a
// time, no blocking, no code shared with the CUDA library.
//
// The paper describes the forward operators only (Section 2, "Computation operators", steps
// 2-4: Logit L = Q K^T, Softmax along the key index, Attend O = A V); what is computed here is
// the chain rule applied to those three steps, for a given gradient dO of the output:
//   step 4 backwards:  dV[j,:] = sum_i A[i,j] dO[i,:]          dA[i,j] = sum_t dO[i,t] V[j,t]
//   step 3 backwards:  dS[i,j] = A[i,j] (dA[i,j] - sum_k A[i,k] dA[i,k])     (softmax Jacobian)
//   step 2 backwards:  dQ[i,:] = scale sum_j dS[i,j] K[j,:]    dK[j,:] = scale sum_i dS[i,j] Q[i,:]
// with S = scale * L the scaled logits.  Masked (query, key) pairs have A = 0 and so take no part;
// a query row without any valid key contributes nothing (its O is 0 by convention, a constant).
// Also returned: lse[i] = log sum_j exp(S[i,j]) over the valid keys (-inf for an empty row), the one
// per-row number from which a backward pass can rebuild A without the row maximum and sum.
//
// Parity pins (tests/test_oracle_bwd_pins.py): central finite differences of the forward oracle,
// long-double brute force with the explicit Jacobian, sum_j dK[j,:] = 0 (key-shift invariance of
// the forward), linearity in dO, closed forms (one key; Q = 0), mask and causal equivalence
// with truncation, lse against an independent log-sum-exp.

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
inline double elem(const void* base, int dtype, int64_t idx) {
    if (dtype == 0) return widen_bf16(static_cast<const uint16_t*>(base)[idx]);
    return static_cast<double>(static_cast<const float*>(base)[idx]);
}

struct Bwd {
    const void *Q, *K, *V, *dO;
    int dtype;
    int64_t B, H, Nq, Nk, d;
    double scale;
    const int32_t* valid_len;
    int causal;
    const int64_t* heads;            // flat (b*H + h) ids, or null = all heads
    int64_t nheads;
    double *dQ, *dK, *dV, *LSE;      // [nheads,Nq,d], [nheads,Nk,d], [nheads,Nk,d], [nheads,Nq] (LSE may be null)
};

// All query rows of one head, one after the other.
void head_bwd(const Bwd& p, int64_t hh) {
    const int64_t bh = p.heads ? p.heads[hh] : hh;
    const int64_t b = bh / p.H;
    const int64_t qoff = bh * p.Nq * p.d, koff = bh * p.Nk * p.d;
    double* dQ = p.dQ + hh * p.Nq * p.d;
    double* dK = p.dK + hh * p.Nk * p.d;
    double* dV = p.dV + hh * p.Nk * p.d;
    for (int64_t x = 0; x < p.Nq * p.d; ++x) dQ[x] = 0.0;
    for (int64_t x = 0; x < p.Nk * p.d; ++x) { dK[x] = 0.0; dV[x] = 0.0; }
    std::vector<double> a(static_cast<size_t>(p.Nk)), dA(static_cast<size_t>(p.Nk));
    for (int64_t i = 0; i < p.Nq; ++i) {
        int64_t n = p.valid_len ? p.valid_len[b] : p.Nk;
        if (p.causal) {
            const int64_t lim = i + 1 + (p.Nk - p.Nq);
            if (lim < n) n = lim;
            if (n < 0) n = 0;
        }
        if (p.LSE) p.LSE[hh * p.Nq + i] = -INFINITY;
        if (n <= 0) continue;
        // forward, steps 2 and 3: scaled logits and their softmax along the keys
        double m = -INFINITY;
        for (int64_t j = 0; j < n; ++j) {
            double acc = 0.0;
            for (int64_t t = 0; t < p.d; ++t)
                acc += elem(p.Q, p.dtype, qoff + i * p.d + t) * elem(p.K, p.dtype, koff + j * p.d + t);
            a[j] = p.scale * acc;
            if (a[j] > m) m = a[j];
        }
        double l = 0.0;
        for (int64_t j = 0; j < n; ++j) { a[j] = std::exp(a[j] - m); l += a[j]; }
        for (int64_t j = 0; j < n; ++j) a[j] /= l;
        if (p.LSE) p.LSE[hh * p.Nq + i] = m + std::log(l);
        // step 4 backwards
        double delta = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            double acc = 0.0;
            for (int64_t t = 0; t < p.d; ++t) {
                const double g = elem(p.dO, p.dtype, qoff + i * p.d + t);
                acc += g * elem(p.V, p.dtype, koff + j * p.d + t);
                dV[j * p.d + t] += a[j] * g;
            }
            dA[j] = acc;
            delta += a[j] * acc;
        }
        // step 3 backwards, then step 2 backwards
        for (int64_t j = 0; j < n; ++j) {
            const double ds = a[j] * (dA[j] - delta);
            for (int64_t t = 0; t < p.d; ++t) {
                dQ[i * p.d + t] += p.scale * ds * elem(p.K, p.dtype, koff + j * p.d + t);
                dK[j * p.d + t] += p.scale * ds * elem(p.Q, p.dtype, qoff + i * p.d + t);
            }
        }
    }
}

void worker(const Bwd* p, int64_t w, int64_t nt) {
    for (int64_t hh = w; hh < p->nheads; hh += nt) head_bwd(*p, hh);
}

}  // namespace

extern "C" int oracle_attn_bwd_heads(const void* Q, const void* K, const void* V, const void* dO, int dtype,
                                     int64_t B, int64_t H, int64_t Nq, int64_t Nk, int64_t d, float scale,
                                     const int32_t* valid_len, int causal, const int64_t* heads, int64_t nheads,
                                     double* dQ, double* dK, double* dV, double* LSE, int nthreads,
                                     int* threads_used) {
    if (!Q || !K || !V || !dO || !dQ || !dK || !dV) return 1;
    if (B < 1 || H < 1 || Nq < 1 || Nk < 1 || d < 1) return 1;
    if (dtype != 0 && dtype != 1) return 1;
    if (!heads) nheads = B * H;
    if (nheads < 0) return 1;
    if (heads) for (int64_t x = 0; x < nheads; ++x) if (heads[x] < 0 || heads[x] >= B * H) return 1;
    if (valid_len) for (int64_t b = 0; b < B; ++b) if (valid_len[b] < 0 || valid_len[b] > Nk) return 1;
    Bwd p{Q, K, V, dO, dtype, B, H, Nq, Nk, d, static_cast<double>(scale), valid_len, causal ? 1 : 0, heads, nheads,
          dQ, dK, dV, LSE};
    int nt = nthreads > 0 ? nthreads : static_cast<int>(std::thread::hardware_concurrency());
    if (nt < 1) nt = 1;
    if (nt > nheads) nt = nheads > 0 ? static_cast<int>(nheads) : 1;
    if (threads_used) *threads_used = nt;
    std::vector<std::thread> pool;
    for (int w = 0; w < nt; ++w) pool.emplace_back(worker, &p, static_cast<int64_t>(w), static_cast<int64_t>(nt));
    for (auto& th : pool) th.join();
    return 0;
}

// fp32 FFMA kernels: the fused attention kernel for any supported dtype/d, and the three
// kernels of the paper's operator-by-operator baseline (Section 4.2, Fig. 7(a)).
//
// All four share one tile shape: 64 query rows x 64 keys per CTA step, 256 threads laid
// out 16 x 16; thread (ty, tx) owns rows ty + 16a and columns tx + 16b, a, b in [0, 4),
// so a row of the logit tile lives in one half-warp and row reductions are four
// shuffle-xor steps.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flat_internal.cuh"

namespace flat {

constexpr int TM = 64;         // query rows per CTA
constexpr int TN = 64;         // keys per step
constexpr int NTHREADS = 256;
constexpr int PSTRIDE = 80;    // padded row stride of the on-chip logit/weight tile

template <typename T> struct Vec16;
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };
template <> struct Vec16<float> { static constexpr int N = 4; };

__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[8]) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}

// Copy rows [row0, row0 + 64) x [0, W) of a row-major [nrows, W] matrix into fp32 shared
// memory with row stride `sstride`; rows past `nrows` are zero-filled.
template <typename T, int W>
__device__ __forceinline__ void load_tile(float* s, int sstride, const T* g, int64_t row0, int64_t nrows) {
    constexpr int N = Vec16<T>::N;
    constexpr int CH = W / N;
    for (int c = threadIdx.x; c < 64 * CH; c += NTHREADS) {
        const int r = c / CH, col = (c % CH) * N;
        float f[N];
        if (row0 + r < nrows) {
            uint4 v = *reinterpret_cast<const uint4*>(g + (row0 + r) * W + col);
            unpack16(v, f);
        } else {
#pragma unroll
            for (int i = 0; i < N; ++i) f[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < N; ++i) s[r * sstride + col + i] = f[i];
    }
}

// acc[a][b] = sum_t Qs[ty + 16a][t] * Ks[tx + 16b][t]  (Logit, Section 2 step 2)
template <int D>
__device__ __forceinline__ void logit_tile(const float* Qs, const float* Ks, float (&acc)[4][4], int ty, int tx) {
    constexpr int S = D + 4;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
#pragma unroll 4
    for (int t = 0; t < D; t += 4) {
        float4 q[4], k[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) q[a] = *reinterpret_cast<const float4*>(Qs + (ty + 16 * a) * S + t);
#pragma unroll
        for (int b = 0; b < 4; ++b) k[b] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * b) * S + t);
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                acc[a][b] = fmaf(q[a].x, k[b].x, acc[a][b]);
                acc[a][b] = fmaf(q[a].y, k[b].y, acc[a][b]);
                acc[a][b] = fmaf(q[a].z, k[b].z, acc[a][b]);
                acc[a][b] = fmaf(q[a].w, k[b].w, acc[a][b]);
            }
    }
}

// o[a][b] += sum_j Ps[ty + 16a][j] * Vs[j][tx + 16b]  (Attend, Section 2 step 4)
template <int D>
__device__ __forceinline__ void attend_tile(const float* Ps, const float* Vs, float (&o)[4][D / 16], int ty, int tx) {
#pragma unroll 2
    for (int j = 0; j < TN; j += 4) {
        float4 p[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) p[a] = *reinterpret_cast<const float4*>(Ps + (ty + 16 * a) * PSTRIDE + j);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            float v[D / 16];
#pragma unroll
            for (int b = 0; b < D / 16; ++b) v[b] = Vs[(j + jj) * D + tx + 16 * b];
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const float pv = jj == 0 ? p[a].x : jj == 1 ? p[a].y : jj == 2 ? p[a].z : p[a].w;
#pragma unroll
                for (int b = 0; b < D / 16; ++b) o[a][b] = fmaf(pv, v[b], o[a][b]);
            }
        }
    }
}

__device__ __forceinline__ float halfwarp_max(float v) {
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float halfwarp_sum(float v) {
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <int D> constexpr size_t fused_smem_bytes() {
    return sizeof(float) * (2 * 64 * (D + 4) + 64 * D + 64 * PSTRIDE);
}

// Fused Logit-Softmax-Attend (Section 5): grid.x = 64-row tiles, grid.y = (b, h).  The
// paper's row-granularity tile would hold all Nk logits of its rows on chip; here the keys
// are streamed 64 at a time with a running row maximum m and sum l, which gives the same
// softmax exactly: sum_j e^{x_j - m'} = e^{m - m'} sum_j e^{x_j - m}.
template <typename T, int D>
__global__ void __launch_bounds__(NTHREADS) fused_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                              const T* __restrict__ V, T* __restrict__ O, int H,
                                                              int Nq, int Nk, float scale_log2e,
                                                              const int32_t* __restrict__ valid_len, int causal,
                                                              float* __restrict__ lse, BiasArg bias) {
    extern __shared__ __align__(16) float smem[];
    float* Qs = smem;
    float* Ks = Qs + 64 * (D + 4);
    float* Vs = Ks + 64 * (D + 4);
    float* Ps = Vs + 64 * D;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t bh = blockIdx.y;
    const int64_t row0 = static_cast<int64_t>(blockIdx.x) * TM;
    int n = valid_len ? min(max(valid_len[bh / H], 0), Nk) : Nk;
    // Causal mask: row r sees keys j < r + 1 + (Nk - Nq); the tile stops at its last row's limit.
    int nrow[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int64_t lim = row0 + ty + 16 * a + 1 + (Nk - Nq);
        nrow[a] = causal ? static_cast<int>(max(static_cast<int64_t>(0), min(static_cast<int64_t>(n), lim))) : n;
    }
    if (causal) n = static_cast<int>(max(static_cast<int64_t>(0), min(static_cast<int64_t>(n), row0 + TM + (Nk - Nq))));
    const T* Qg = Q + bh * Nq * D;
    const T* Kg = K + bh * Nk * D;
    const T* Vg = V + bh * Nk * D;

    load_tile<T, D>(Qs, D + 4, Qg, row0, Nq);

    float m[4], l[4], o[4][D / 16];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        m[a] = -INFINITY; l[a] = 0.f;
#pragma unroll
        for (int b = 0; b < D / 16; ++b) o[a][b] = 0.f;
    }

    for (int k0 = 0; k0 < n; k0 += TN) {
        __syncthreads();
        load_tile<T, D>(Ks, D + 4, Kg, k0, n);
        load_tile<T, D>(Vs, D, Vg, k0, n);
        __syncthreads();
        float s[4][4];
        logit_tile<D>(Qs, Ks, s, ty, tx);
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float mx = -INFINITY;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                s[a][b] = (k0 + tx + 16 * b < nrow[a]) ? s[a][b] * scale_log2e : -INFINITY;
                // additive bias of the scaled logit (natural units -> base 2); -inf switches the pair off
                if (bias.p && k0 + tx + 16 * b < nrow[a] && row0 + ty + 16 * a < Nq) {
                    const long long at = (bh / H) * bias.sb + (bh % H) * bias.sh + (row0 + ty + 16 * a) * Nk + k0 + tx + 16 * b;
                    const float bv = bias.f32 ? static_cast<const float*>(bias.p)[at]
                                              : __bfloat162float(static_cast<const __nv_bfloat16*>(bias.p)[at]);
                    s[a][b] = fmaf(bv, 1.4426950408889634f, s[a][b]);
                }
                mx = fmaxf(mx, s[a][b]);
            }
            mx = halfwarp_max(mx);
            const float m_new = fmaxf(m[a], mx);
            // (a row that has seen no valid key yet -- possible under the causal mask -- keeps m = -inf;
            // the reference below is then 0, so that its weights and alpha come out as 0 and not NaN)
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            const float alpha = exp2f(m[a] - m_use);   // exp2(-inf) = 0 on the first tile
            float sum = 0.f;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const float p = exp2f(s[a][b] - m_use);
                sum += p;
                Ps[(ty + 16 * a) * PSTRIDE + tx + 16 * b] = p;
            }
            l[a] = l[a] * alpha + halfwarp_sum(sum);
            m[a] = m_new;
#pragma unroll
            for (int b = 0; b < D / 16; ++b) o[a][b] *= alpha;
        }
        __syncthreads();
        attend_tile<D>(Ps, Vs, o, ty, tx);
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int64_t r = row0 + ty + 16 * a;
        if (r >= Nq) continue;
        const float inv = l[a] > 0.f ? 1.f / l[a] : 0.f;   // no valid key: O = 0
#pragma unroll
        for (int b = 0; b < D / 16; ++b) store_out(O + (bh * Nq + r) * D + tx + 16 * b, o[a][b] * inv);
        // log of the row's sum of exponentials (m and the exponents are in base-2 units here)
        if (lse && tx == 0) lse[bh * Nq + r] = l[a] > 0.f ? (m[a] + log2f(l[a])) * 0.6931471805599453f : -INFINITY;
    }
}

// Baseline kernel 1: L = scale * Q K^T, written to device memory (fp32).
template <typename T, int D>
__global__ void __launch_bounds__(NTHREADS) naive_logit_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                               float* __restrict__ L, int Nq, int Nk, float scale) {
    extern __shared__ __align__(16) float smem[];
    float* Qs = smem;
    float* Ks = Qs + 64 * (D + 4);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t bh = blockIdx.z;
    const int64_t row0 = static_cast<int64_t>(blockIdx.y) * TM, k0 = static_cast<int64_t>(blockIdx.x) * TN;
    load_tile<T, D>(Qs, D + 4, Q + bh * Nq * D, row0, Nq);
    load_tile<T, D>(Ks, D + 4, K + bh * Nk * D, k0, Nk);
    __syncthreads();
    float s[4][4];
    logit_tile<D>(Qs, Ks, s, ty, tx);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int64_t r = row0 + ty + 16 * a;
        if (r >= Nq) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int64_t c = k0 + tx + 16 * b;
            if (c < Nk) L[(bh * Nq + r) * Nk + c] = s[a][b] * scale;
        }
    }
}

// Baseline kernel 2: A = softmax of each row of L over the valid keys.  One CTA per row;
// pass 1 finds (max, sum) in one sweep, pass 2 re-reads the row and writes the weights.
template <typename TA>
__global__ void __launch_bounds__(NTHREADS) naive_softmax_kernel(const float* __restrict__ L, TA* __restrict__ A,
                                                                 int H, int Nq, int Nk,
                                                                 const int32_t* __restrict__ valid_len, int causal) {
    __shared__ float red_m[NTHREADS / 32], red_l[NTHREADS / 32];
    const int64_t row = blockIdx.x;
    int n = valid_len ? min(max(valid_len[(row / Nq) / H], 0), Nk) : Nk;
    if (causal) n = static_cast<int>(max(static_cast<int64_t>(0), min(static_cast<int64_t>(n), row % Nq + 1 + (Nk - Nq))));
    const float* Lr = L + row * Nk;
    TA* Ar = A + row * Nk;
    constexpr float LOG2E = 1.4426950408889634f;
    float m = -INFINITY, l = 0.f;
    for (int j = threadIdx.x; j < n; j += NTHREADS) {
        const float x = Lr[j] * LOG2E;
        if (x > m) { l *= exp2f(m - x); m = x; }
        l += exp2f(x - m);
    }
    // combine (m, l) pairs: warp, then CTA
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
        const float mm = fmaxf(m, m2);
        l = (m == -INFINITY ? 0.f : l * exp2f(m - mm)) + (m2 == -INFINITY ? 0.f : l2 * exp2f(m2 - mm));
        m = mm;
    }
    if ((threadIdx.x & 31) == 0) { red_m[threadIdx.x >> 5] = m; red_l[threadIdx.x >> 5] = l; }
    __syncthreads();
    m = red_m[0]; l = 0.f;
#pragma unroll
    for (int w = 1; w < NTHREADS / 32; ++w) m = fmaxf(m, red_m[w]);
#pragma unroll
    for (int w = 0; w < NTHREADS / 32; ++w) l += red_m[w] == -INFINITY ? 0.f : red_l[w] * exp2f(red_m[w] - m);
    const float inv = l > 0.f ? 1.f / l : 0.f;
    for (int j = threadIdx.x; j < Nk; j += NTHREADS)
        store_out(Ar + j, j < n ? exp2f(Lr[j] * LOG2E - m) * inv : 0.f);
}

// Baseline kernel 3: O = A V.
template <typename T, typename TA, int D>
__global__ void __launch_bounds__(NTHREADS) naive_attend_kernel(const TA* __restrict__ A, const T* __restrict__ V,
                                                                T* __restrict__ O, int H, int Nq, int Nk,
                                                                const int32_t* __restrict__ valid_len) {
    extern __shared__ __align__(16) float smem[];
    float* Vs = smem;
    float* Ps = Vs + 64 * D;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int64_t bh = blockIdx.y;
    const int64_t row0 = static_cast<int64_t>(blockIdx.x) * TM;
    const int n = valid_len ? min(max(valid_len[bh / H], 0), Nk) : Nk;
    const TA* Ag = A + bh * Nq * Nk;
    float o[4][D / 16];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < D / 16; ++b) o[a][b] = 0.f;
    for (int k0 = 0; k0 < n; k0 += TN) {
        __syncthreads();
        load_tile<T, D>(Vs, D, V + bh * Nk * D, k0, n);
        for (int c = threadIdx.x; c < 64 * 64; c += NTHREADS) {
            const int r = c >> 6, j = c & 63;
            float p = 0.f;
            if (row0 + r < Nq && k0 + j < n) p = static_cast<float>(Ag[(row0 + r) * Nk + k0 + j]);
            Ps[r * PSTRIDE + j] = p;
        }
        __syncthreads();
        attend_tile<D>(Ps, Vs, o, ty, tx);
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int64_t r = row0 + ty + 16 * a;
        if (r >= Nq) continue;
#pragma unroll
        for (int b = 0; b < D / 16; ++b) store_out(O + (bh * Nq + r) * D + tx + 16 * b, o[a][b]);
    }
}

template <typename T, int D>
static int launch_fused_simt_td(const Problem& p, cudaStream_t st) {
    auto kern = fused_simt_kernel<T, D>;
    const size_t smem = fused_smem_bytes<D>();
    if (!ensure_dynamic_smem<fused_simt_kernel<T, D>>(smem)) return FLAT_ERR_CUDA;
    dim3 grid((p.Nq + TM - 1) / TM, p.B * p.H);
    kern<<<grid, NTHREADS, smem, st>>>(static_cast<const T*>(p.Q), static_cast<const T*>(p.K),
                                       static_cast<const T*>(p.V), static_cast<T*>(p.O), p.H, p.Nq, p.Nk,
                                       p.scale * 1.4426950408889634f, p.k_valid_len, p.causal, p.lse, bias_arg(p));
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

template <typename T, typename TA, int D>
static int launch_naive_td(const Problem& p, float* L, void* A, cudaStream_t st) {
    {
        auto kern = naive_logit_kernel<T, D>;
        const size_t smem = sizeof(float) * 2 * 64 * (D + 4);
        if (!ensure_dynamic_smem<naive_logit_kernel<T, D>>(smem)) return FLAT_ERR_CUDA;
        dim3 grid((p.Nk + TN - 1) / TN, (p.Nq + TM - 1) / TM, p.B * p.H);
        kern<<<grid, NTHREADS, smem, st>>>(static_cast<const T*>(p.Q), static_cast<const T*>(p.K), L, p.Nq, p.Nk,
                                           p.scale);
        if (cudaGetLastError() != cudaSuccess) return FLAT_ERR_CUDA;
    }
    {
        const int64_t rows = static_cast<int64_t>(p.B) * p.H * p.Nq;
        naive_softmax_kernel<TA><<<static_cast<unsigned>(rows), NTHREADS, 0, st>>>(L, static_cast<TA*>(A), p.H, p.Nq,
                                                                                   p.Nk, p.k_valid_len, p.causal);
        if (cudaGetLastError() != cudaSuccess) return FLAT_ERR_CUDA;
    }
    {
        auto kern = naive_attend_kernel<T, TA, D>;
        const size_t smem = sizeof(float) * (64 * D + 64 * PSTRIDE);
        if (!ensure_dynamic_smem<naive_attend_kernel<T, TA, D>>(smem)) return FLAT_ERR_CUDA;
        dim3 grid((p.Nq + TM - 1) / TM, p.B * p.H);
        kern<<<grid, NTHREADS, smem, st>>>(static_cast<const TA*>(A), static_cast<const T*>(p.V),
                                           static_cast<T*>(p.O), p.H, p.Nq, p.Nk, p.k_valid_len);
        if (cudaGetLastError() != cudaSuccess) return FLAT_ERR_CUDA;
    }
    return FLAT_OK;
}

template <typename T>
static int launch_fused_simt_t(const Problem& p, cudaStream_t st) {
    switch (p.d) {
        case 16: return launch_fused_simt_td<T, 16>(p, st);
        case 32: return launch_fused_simt_td<T, 32>(p, st);
        case 64: return launch_fused_simt_td<T, 64>(p, st);
        case 128: return launch_fused_simt_td<T, 128>(p, st);
    }
    return FLAT_ERR_UNSUPPORTED;
}

int launch_fused_simt(const Problem& p, cudaStream_t st) {
    return p.dtype == FLAT_DTYPE_BF16 ? launch_fused_simt_t<__nv_bfloat16>(p, st) : launch_fused_simt_t<float>(p, st);
}

int launch_naive(const Problem& p, void* L, void* A, cudaStream_t st) {
    float* Lf = static_cast<float*>(L);
    if (naive_tc_applies(p)) {
        // contractions on the tensor cores, row softmax between them as below
        int rc = launch_naive_logit_tc(p, Lf, st);
        if (rc != FLAT_OK) return rc;
        const int64_t rows = static_cast<int64_t>(p.B) * p.H * p.Nq;
        naive_softmax_kernel<__nv_bfloat16><<<static_cast<unsigned>(rows), NTHREADS, 0, st>>>(
            Lf, static_cast<__nv_bfloat16*>(A), p.H, p.Nq, p.Nk, p.k_valid_len, p.causal);
        if (cudaGetLastError() != cudaSuccess) return FLAT_ERR_CUDA;
        return launch_naive_attend_tc(p, A, st);
    }
    if (p.dtype == FLAT_DTYPE_BF16) {
        switch (p.d) {
            case 16: return launch_naive_td<__nv_bfloat16, __nv_bfloat16, 16>(p, Lf, A, st);
            case 32: return launch_naive_td<__nv_bfloat16, __nv_bfloat16, 32>(p, Lf, A, st);
            case 64: return launch_naive_td<__nv_bfloat16, __nv_bfloat16, 64>(p, Lf, A, st);
            case 128: return launch_naive_td<__nv_bfloat16, __nv_bfloat16, 128>(p, Lf, A, st);
        }
    } else {
        switch (p.d) {
            case 16: return launch_naive_td<float, float, 16>(p, Lf, A, st);
            case 32: return launch_naive_td<float, float, 32>(p, Lf, A, st);
            case 64: return launch_naive_td<float, float, 64>(p, Lf, A, st);
            case 128: return launch_naive_td<float, float, 128>(p, Lf, A, st);
        }
    }
    return FLAT_ERR_UNSUPPORTED;
}

}  // namespace flat

// The normalisation layer of an attention block (paper Section 2: a block is an attention layer, a
// normalisation layer and fully connected layers; the paper does not say which normalisation).
// Reading taken: layer normalisation over the feature index of each token, after the residual add,
//     z = x + r (r optional),   y = gamma * (z - mean(z)) / sqrt(var(z) + eps) + beta,
// with the biased variance, bf16 storage and fp32 statistics.
//
// Bound: device-memory bandwidth -- every element of x (and r) is read once and y written once, so
// the algorithmic traffic is 2 bytes * M * D * (2 or 3).  One warp per row of up to 1024 features (2, 4
// or 8 warps for longer rows): the row is read with 16-byte loads (a warp covers 512 contiguous bytes per
// load instruction), kept in registers, reduced with shuffles (two passes over the registers: mean, then
// centred sum of squares), normalised and written back with 16-byte stores.  Rows are dealt to the CTAs
// of a grid sized to the SM count.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flat_internal.cuh"

namespace flat {

namespace {

constexpr int LN_WARPS = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { f[2 * e] = __uint_as_float(w[e] << 16); f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
}
__device__ __forceinline__ uint32_t pack2bf(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// WPR warps share a row (1, 2, 4 or 8: rows of more than 1024 features are split so that a lane holds at
// most four vectors); NV: vectors per lane.  The CTA's eight warps work on 8 / WPR rows at a time.
template <int NV, int WPR, bool RES>
__global__ void __launch_bounds__(LN_WARPS * 32)
layernorm_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ R,
                 const __nv_bfloat16* __restrict__ gamma, const __nv_bfloat16* __restrict__ beta,
                 __nv_bfloat16* __restrict__ Y, long long M, int D, float eps) {
    constexpr int RPB = LN_WARPS / WPR;                   // rows per CTA and iteration
    __shared__ float red[2][2][LN_WARPS];                 // [iteration parity][sum | squares][warp]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wr = warp / WPR, wp = warp % WPR;           // row of the CTA's group, part of the row
    const int nvec = D >> 3;                              // 16-byte vectors per row
    const float inv_d = 1.f / static_cast<float>(D);
    int it = 0;
    for (long long row0 = static_cast<long long>(blockIdx.x) * RPB; row0 < M; row0 += static_cast<long long>(gridDim.x) * RPB, it ^= 1) {
        const long long row = row0 + wr;
        const bool live = row < M;
        const uint4* x = reinterpret_cast<const uint4*>(X + row * D);
        const uint4* r = RES ? reinterpret_cast<const uint4*>(R + row * D) : nullptr;
        float z[NV][8];
        float sum = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = (v * WPR + wp) * 32 + lane;
            if (live && idx < nvec) {
                unpack8(x[idx], z[v]);
                if (RES) {
                    float rr[8];
                    unpack8(r[idx], rr);
#pragma unroll
                    for (int e = 0; e < 8; ++e) z[v][e] += rr[e];
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) sum += z[v][e];
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) z[v][e] = 0.f;
            }
        }
        sum = warp_sum(sum);
        if (WPR > 1) {
            if (lane == 0) red[it][0][warp] = sum;
            __syncthreads();
            sum = 0.f;
#pragma unroll
            for (int p = 0; p < WPR; ++p) sum += red[it][0][wr * WPR + p];
        }
        const float mean = sum * inv_d;
        float sq = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (live && (v * WPR + wp) * 32 + lane < nvec) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { const float c = z[v][e] - mean; sq = fmaf(c, c, sq); }
            }
        }
        sq = warp_sum(sq);
        if (WPR > 1) {
            if (lane == 0) red[it][1][warp] = sq;
            __syncthreads();
            sq = 0.f;
#pragma unroll
            for (int p = 0; p < WPR; ++p) sq += red[it][1][wr * WPR + p];
        }
        const float rstd = rsqrtf(sq * inv_d + eps);
        uint4* y = reinterpret_cast<uint4*>(Y + row * D);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = (v * WPR + wp) * 32 + lane;
            if (live && idx < nvec) {
                float g[8], b[8];
                unpack8(reinterpret_cast<const uint4*>(gamma)[idx], g);
                unpack8(reinterpret_cast<const uint4*>(beta)[idx], b);
                uint4 o;
                o.x = pack2bf(fmaf((z[v][0] - mean) * rstd, g[0], b[0]), fmaf((z[v][1] - mean) * rstd, g[1], b[1]));
                o.y = pack2bf(fmaf((z[v][2] - mean) * rstd, g[2], b[2]), fmaf((z[v][3] - mean) * rstd, g[3], b[3]));
                o.z = pack2bf(fmaf((z[v][4] - mean) * rstd, g[4], b[4]), fmaf((z[v][5] - mean) * rstd, g[5], b[5]));
                o.w = pack2bf(fmaf((z[v][6] - mean) * rstd, g[6], b[6]), fmaf((z[v][7] - mean) * rstd, g[7], b[7]));
                y[idx] = o;
            }
        }
    }
}

template <int NV, int WPR>
int launch_ln_nv(const void* X, const void* R, const void* gamma, const void* beta, void* Y, long long M, int D,
                 float eps, cudaStream_t st) {
    constexpr int RPB = LN_WARPS / WPR;
    const long long blocks_needed = (M + RPB - 1) / RPB;
    const long long cap = static_cast<long long>(device_sm_count()) * 8;      // 8 CTAs of 256 threads per SM
    const int grid = static_cast<int>(blocks_needed < cap ? blocks_needed : cap);
    auto bf = [](const void* p) { return static_cast<const __nv_bfloat16*>(p); };
    if (R) layernorm_kernel<NV, WPR, true><<<grid, LN_WARPS * 32, 0, st>>>(bf(X), bf(R), bf(gamma), bf(beta), static_cast<__nv_bfloat16*>(Y), M, D, eps);
    else   layernorm_kernel<NV, WPR, false><<<grid, LN_WARPS * 32, 0, st>>>(bf(X), nullptr, bf(gamma), bf(beta), static_cast<__nv_bfloat16*>(Y), M, D, eps);
    return cudaGetLastError() == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

}  // namespace

int launch_layernorm(const void* X, const void* R, const void* gamma, const void* beta, void* Y, long long M, int D,
                     float eps, cudaStream_t st) {
    const int nv = (D / 8 + 31) / 32;                     // vectors per lane if one warp took the row
    if (nv <= 1) return launch_ln_nv<1, 1>(X, R, gamma, beta, Y, M, D, eps, st);
    if (nv <= 2) return launch_ln_nv<2, 1>(X, R, gamma, beta, Y, M, D, eps, st);
    if (nv <= 4) return launch_ln_nv<4, 1>(X, R, gamma, beta, Y, M, D, eps, st);
    if (nv <= 8) return launch_ln_nv<4, 2>(X, R, gamma, beta, Y, M, D, eps, st);
    if (nv <= 16) return launch_ln_nv<4, 4>(X, R, gamma, beta, Y, M, D, eps, st);
    if (nv <= 32) return launch_ln_nv<4, 8>(X, R, gamma, beta, Y, M, D, eps, st);
    return FLAT_ERR_UNSUPPORTED;
}

}  // namespace flat

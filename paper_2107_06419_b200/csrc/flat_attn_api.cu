// C ABI of libflat_attn: argument validation and dispatch.  No kernel code here.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <mutex>

#include "flat_internal.cuh"

namespace {

thread_local int g_last_launches = 0;
thread_local int g_last_variant = 0;

// The library's own device status word: kernels that give up on a bounded wait store their code
// here when the caller passed no `status` word, so that a timeout always leaves a trace.  In host
// code the name is a handle for the runtime's symbol table; its device address is looked up once
// per device.
__device__ int32_t g_device_error = 0;
constexpr int kMaxDevices = 64;
std::mutex g_err_mu;
int32_t* g_err_addr[kMaxDevices];
bool g_err_ready[kMaxDevices];

int32_t* library_status_word() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_err_mu);
    if (!g_err_ready[dev]) {
        void* a = nullptr;
        if (cudaGetSymbolAddress(&a, g_device_error) != cudaSuccess || a == nullptr) {
            cudaGetLastError();                          // (no device, or no image for it: the caller's launch will say so)
            return nullptr;
        }
        g_err_addr[dev] = static_cast<int32_t*>(a);
        g_err_ready[dev] = true;
    }
    return g_err_addr[dev];
}
inline int32_t* status_or_library_word(int32_t* s) { return s ? s : library_status_word(); }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate(const flat_attn_params_t* p, flat::Problem* out) {
    if (!p) return FLAT_ERR_NULL;
    if (!p->Q || !p->K || !p->V || !p->O) return FLAT_ERR_NULL;
    if (p->B < 1 || p->H < 1 || p->Nq < 1 || p->Nk < 1 || p->d < 1) return FLAT_ERR_SHAPE;
    if (!isfinite(p->scale)) return FLAT_ERR_SHAPE;
    const int64_t bh = static_cast<int64_t>(p->B) * p->H;
    if (bh > 65535) return FLAT_ERR_SHAPE;
    // B*H*Nq*Nk < 2^16 * 2^31 * 2^31 could overflow 63 bits: check stepwise.
    const int64_t lim = INT64_MAX / 16;
    if (bh * p->Nq > lim / p->Nk) return FLAT_ERR_SHAPE;
    if (bh * static_cast<int64_t>(p->Nq > p->Nk ? p->Nq : p->Nk) > lim / p->d) return FLAT_ERR_SHAPE;
    if (p->dtype != FLAT_DTYPE_BF16 && p->dtype != FLAT_DTYPE_F32) return FLAT_ERR_UNSUPPORTED;
    if (p->d != 16 && p->d != 32 && p->d != 64 && p->d != 128) return FLAT_ERR_UNSUPPORTED;
    if (p->variant < FLAT_VARIANT_AUTO || p->variant > FLAT_VARIANT_TC2_HALVES_SPLIT16) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(p->Q) || !aligned16(p->K) || !aligned16(p->V) || !aligned16(p->O)) return FLAT_ERR_ALIGN;
    if (p->k_valid_len && (reinterpret_cast<uintptr_t>(p->k_valid_len) & 3u)) return FLAT_ERR_ALIGN;
    if (p->status && (reinterpret_cast<uintptr_t>(p->status) & 3u)) return FLAT_ERR_ALIGN;
    if (p->causal != 0 && p->causal != 1) return FLAT_ERR_UNSUPPORTED;
    if (p->lse && (reinterpret_cast<uintptr_t>(p->lse) & 3u)) return FLAT_ERR_ALIGN;
    if (p->bias) {
        if (p->bias_dtype != FLAT_DTYPE_BF16 && p->bias_dtype != FLAT_DTYPE_F32) return FLAT_ERR_UNSUPPORTED;
        if (p->bias_stride_b < 0 || p->bias_stride_h < 0) return FLAT_ERR_SHAPE;
        if (reinterpret_cast<uintptr_t>(p->bias) & (p->bias_dtype == FLAT_DTYPE_F32 ? 3u : 1u)) return FLAT_ERR_ALIGN;
    }
    if (p->block_mask && (p->block_mask_stride_b < 0 || p->block_mask_stride_h < 0)) return FLAT_ERR_SHAPE;
    *out = flat::Problem{p->Q, p->K, p->V, p->O, p->B, p->H, p->Nq, p->Nk, p->d,
                         p->scale, p->dtype, p->k_valid_len, status_or_library_word(p->status), p->causal, p->lse,
                         p->bias, p->bias_dtype, p->bias_stride_b, p->bias_stride_h,
                         p->block_mask, p->block_mask_stride_b, p->block_mask_stride_h};
    return FLAT_OK;
}

}  // namespace

namespace flat {
int check_params(const flat_attn_params_t* p) {
    Problem q;
    return validate(p, &q);
}
}  // namespace flat

namespace {

bool tc_applies(const flat::Problem& q) {
    return q.dtype == FLAT_DTYPE_BF16 && (q.d == 64 || q.d == 128);
}

int run_fused(const flat::Problem& q, int variant, cudaStream_t st) {
    int v = variant;
    if (v == FLAT_VARIANT_AUTO) {
        if (!tc_applies(q)) {
            // fp32 tensors: the split-tf32 tensor-core kernel where it applies, else the FFMA kernel
            v = flat::tf32_applies(q) ? FLAT_VARIANT_TF32 : FLAT_VARIANT_SIMT;
        } else {
            // Two-tile CTAs (256 query rows) once they fill the SMs; otherwise 128-row CTAs, which
            // give twice as many CTAs for small problems.  At d = 64 the two-tile kernel is the one
            // with two softmax threads per row (measured 15-20 % faster than TC2 on every d = 64
            // workload), and it is taken as soon as half the SMs get a CTA.
            const int64_t ctas2 = static_cast<int64_t>((q.Nq + 255) / 256) * q.B * q.H;
            const int sms = flat::device_sm_count();
            // (with eight key steps or fewer a CTA is mostly fill and drain: two single-tile CTAs per SM
            // overlap each other's, measured 3-14 % ahead of the two-tile kernel there)
            // ... unless the two-tile kernel gets at least two items per SM: it then runs its persistent
            // grid, where fill and drain are paid once per CTA instead of once per item (measured 11-26 %
            // ahead of the single-tile CTAs at 512 and 1024 keys).
            // (not when the 256-row slabs would be more than a quarter padding, e.g. 128 query rows)
            if (q.d == 64) {
                const bool slabs_fill = 3 * 256 * static_cast<int64_t>((q.Nq + 255) / 256) <= 4 * static_cast<int64_t>(q.Nq);
                v = ((2 * ctas2 >= sms && q.Nk > 1024) || (ctas2 >= 2 * sms && !q.k_valid_len && slabs_fill))
                        ? FLAT_VARIANT_TC3 : FLAT_VARIANT_TC2_SINGLE;
            }
            // d = 128: the two-tile kernel (lazy reference maximum, polynomial exp2, packed arithmetic)
            // is ahead of its single-tile predecessor even when it leaves SMs empty (B2 H8 2048 keys:
            // 0.037 against 0.096 ms); only tiny problems (256 keys or fewer, less than one CTA per SM)
            // are at par or a few per cent better on the 128-row CTAs.
            else           v = (ctas2 >= sms || q.Nk > 256) ? FLAT_VARIANT_TC2 : FLAT_VARIANT_TC;
            // (the single-tile predecessor kernel has no causal mask and does not write lse)
            if ((q.causal || q.lse) && v == FLAT_VARIANT_TC) v = FLAT_VARIANT_TC2;
            // (the bias is read by the two-tile kernel with one thread per row)
            if (q.bias) v = FLAT_VARIANT_TC2;
            // (pruned attention runs on the one-tile kernel: a CTA walks the list of its query tile's kept key tiles)
            if (q.block_mask) v = FLAT_VARIANT_TC2_SINGLE;
            // A launch of single-tile CTAs that would leave most SMs empty splits the keys of every query tile
            // over a cluster of 8, 4 or 2 CTAs: the per-CTA chain of key steps, which is what such a launch waits
            // for, gets that much shorter at the price of one exchange through distributed shared memory (1-2 us).
            // The largest split that still fits the GPU at two CTAs per SM and leaves every CTA two key steps
            // (one is enough while every CTA gets an SM of its own).
            if (v == FLAT_VARIANT_TC2_SINGLE && q.d == 64 && !q.block_mask && !q.bias) {
                const int64_t ctas1 = static_cast<int64_t>((q.Nq + 127) / 128) * q.B * q.H;
                const int key_tiles = (q.Nk + 127) / 128;
                for (int cs = 8; cs >= 2; cs /= 2) {
                    if (ctas1 * cs > 7 * sms / 4) continue;
                    if (key_tiles < (ctas1 * cs <= sms ? cs : 2 * cs)) continue;
                    v = cs == 8 ? FLAT_VARIANT_TC2_SPLIT8 : cs == 4 ? FLAT_VARIANT_TC2_SPLIT4 : FLAT_VARIANT_TC2_SPLIT2;
                    break;
                }
                // While every CTA gets an SM of its own, the tile is better worked on by two warpgroups that take
                // alternate key tiles (half the chain again, no exchange between CTAs for that half): the largest
                // cluster that leaves each warpgroup a key tile and fits -- eight-CTA clusters of one-per-SM CTAs
                // only up to half the SMs, beyond that they no longer all start at once (measured on 16 tiles x
                // 16 key tiles: 17.1 us against 9.6 with clusters of four).
                for (int cs = 16; cs >= 1 && key_tiles >= 2; cs /= 2) {
                    if (ctas1 * cs > (cs >= 8 ? sms / 2 : 7 * sms / 8)) continue;
                    if (key_tiles < 2 * cs) continue;
                    if (cs == 16 && ctas1 > 2) continue;     // (clusters of sixteen: for one or two query tiles, see d = 128 below)
                    v = cs == 16 ? FLAT_VARIANT_TC2_HALVES_SPLIT16 : cs == 8 ? FLAT_VARIANT_TC2_HALVES_SPLIT8 : cs == 4 ? FLAT_VARIANT_TC2_HALVES_SPLIT4
                        : cs == 2 ? FLAT_VARIANT_TC2_HALVES_SPLIT2 : FLAT_VARIANT_TC2_HALVES;
                    break;
                }
            }
            // d = 128: the same split (one CTA per SM there: 160 KB of tiles) while the two-tile CTAs would cover
            // less than half the SMs and every CTA of the split keeps at least two key steps (128 queries x
            // 16K keys, 8 heads: 247 -> 41 us).
            if (q.d == 128 && !q.block_mask && !q.bias && 2 * ctas2 < sms) {
                const int64_t ctas1 = static_cast<int64_t>((q.Nq + 127) / 128) * q.B * q.H;
                const int key_tiles = (q.Nk + 127) / 128;
                for (int cs = 16; cs >= 2; cs /= 2) {
                    if (ctas1 * cs > sms || key_tiles < 2 * cs) continue;
                    // (clusters of sixteen -- beyond the portable size -- pay for one or two query tiles only: 128
                    // queries x 64K keys 123 -> 83 us, two heads x 32K keys 68 -> 55 us; with three or four clusters
                    // they are at par with eight, with eight clusters twice as slow)
                    if (cs == 16 && ctas1 > 2) continue;
                    v = cs == 16 ? FLAT_VARIANT_TC2_SPLIT16 : cs == 8 ? FLAT_VARIANT_TC2_SPLIT8
                        : cs == 4 ? FLAT_VARIANT_TC2_SPLIT4 : FLAT_VARIANT_TC2_SPLIT2;
                    break;
                }
            }
        }
    }
    if (q.causal && v == FLAT_VARIANT_TC) return FLAT_ERR_UNSUPPORTED;
    if (q.lse && (v == FLAT_VARIANT_TC || v == FLAT_VARIANT_RGRAN)) return FLAT_ERR_UNSUPPORTED;
    if (q.bias && v != FLAT_VARIANT_TC2 && v != FLAT_VARIANT_SIMT) return FLAT_ERR_UNSUPPORTED;
    if ((v >= FLAT_VARIANT_TC2_HALVES && v <= FLAT_VARIANT_TC2_HALVES_SPLIT8) || v == FLAT_VARIANT_TC2_HALVES_SPLIT16) {
        if (!tc_applies(q) || q.d != 64 || q.block_mask || q.bias) return FLAT_ERR_UNSUPPORTED;
        const int cs = v == FLAT_VARIANT_TC2_HALVES_SPLIT16 ? 16 : 1 << (v - FLAT_VARIANT_TC2_HALVES);
        int rc = flat::launch_fused_tc2_halves(q, st, cs, variant == FLAT_VARIANT_AUTO);
        if (rc != FLAT_OK && cs == 16 && variant == FLAT_VARIANT_AUTO) {
            // (AUTO asked for sixteen and the device cannot hold all the launch's clusters at once, or refused the
            // launch: eight)
            cudaGetLastError();
            v = FLAT_VARIANT_TC2_HALVES_SPLIT8;
            rc = flat::launch_fused_tc2_halves(q, st, 8);
        }
        g_last_variant = v;
        return rc;
    }
    if (v == FLAT_VARIANT_TC2_SPLIT2 || v == FLAT_VARIANT_TC2_SPLIT4 || v == FLAT_VARIANT_TC2_SPLIT8 || v == FLAT_VARIANT_TC2_SPLIT16) {
        if (!tc_applies(q) || q.block_mask || (v == FLAT_VARIANT_TC2_SPLIT16 && q.d != 128)) return FLAT_ERR_UNSUPPORTED;
        const int cs = v == FLAT_VARIANT_TC2_SPLIT2 ? 2 : v == FLAT_VARIANT_TC2_SPLIT4 ? 4 : v == FLAT_VARIANT_TC2_SPLIT8 ? 8 : 16;
        int rc = flat::launch_fused_tc2_single(q, st, cs, variant == FLAT_VARIANT_AUTO);
        if (rc != FLAT_OK && cs == 16 && variant == FLAT_VARIANT_AUTO) {
            // (AUTO asked for sixteen and the device cannot hold all the launch's clusters at once, or refused the
            // launch: eight)
            cudaGetLastError();
            v = FLAT_VARIANT_TC2_SPLIT8;
            rc = flat::launch_fused_tc2_single(q, st, 8);
        }
        g_last_variant = v;
        return rc;
    }
    if (v == FLAT_VARIANT_TF32 && !flat::tf32_applies(q)) return FLAT_ERR_UNSUPPORTED;
    if (q.block_mask && (v != FLAT_VARIANT_TC2_SINGLE || q.bias || !tc_applies(q) || q.Nk > 131072)) return FLAT_ERR_UNSUPPORTED;
    g_last_variant = v;
    if (v == FLAT_VARIANT_TC2_SINGLE) {
        if (!tc_applies(q) || (q.d != 64 && !q.block_mask)) return FLAT_ERR_UNSUPPORTED;
        return flat::launch_fused_tc2_single(q, st);
    }
    if (v == FLAT_VARIANT_TC3) {
        if (!tc_applies(q) || q.d != 64) return FLAT_ERR_UNSUPPORTED;
        return flat::launch_fused_tc3(q, st);
    }
    if (v == FLAT_VARIANT_TF32) return flat::launch_fused_tf32(q, st);
    if (v == FLAT_VARIANT_RGRAN) return flat::launch_fused_rgran(q, st);   // (checks its own conditions)
    if (v == FLAT_VARIANT_TC || v == FLAT_VARIANT_TC2) {
        if (!tc_applies(q)) return FLAT_ERR_UNSUPPORTED;
        return v == FLAT_VARIANT_TC ? flat::launch_fused_tc(q, st) : flat::launch_fused_tc2(q, st);
    }
    return flat::launch_fused_simt(q, st);
}

inline size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// Side streams and events of flat_attn_fwd_host, one set per device and host thread, created on
// first use and kept until the process exits.
struct HostPipe {
    cudaStream_t side[2];
    cudaEvent_t fork, join[2];
};

HostPipe* host_pipe() {
    thread_local HostPipe pipes[16];
    thread_local bool ready[16] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) return nullptr;
    if (!ready[dev]) {
        HostPipe& h = pipes[dev];
        if (cudaStreamCreateWithFlags(&h.side[0], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&h.side[1], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&h.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&h.join[0], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&h.join[1], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        ready[dev] = true;
    }
    return &pipes[dev];
}

}  // namespace

extern "C" {

int flat_attn_fwd_ex(const flat_attn_params_t* p, void* stream) {
    flat::Problem q;
    const int rc = validate(p, &q);
    if (rc != FLAT_OK) return rc;
    const int r = run_fused(q, p->variant, static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_attn_fwd(const void* Q, const void* K, const void* V, void* O, int B, int H, int Nq, int Nk, int d,
                  float scale, void* stream) {
    flat_attn_params_t p{Q, K, V, O, B, H, Nq, Nk, d, scale, FLAT_DTYPE_BF16, nullptr, nullptr, FLAT_VARIANT_AUTO, 0, nullptr, nullptr, 0, 0, 0, nullptr, 0, 0};
    return flat_attn_fwd_ex(&p, stream);
}

int flat_attn_naive_fwd_ex(const flat_attn_params_t* p, void* L, void* A, void* stream) {
    flat::Problem q;
    const int rc = validate(p, &q);
    if (rc != FLAT_OK) return rc;
    if (!L || !A) return FLAT_ERR_NULL;
    if (q.bias || q.block_mask) return FLAT_ERR_UNSUPPORTED; // (the baseline has no bias operand and no pruning map)
    if (!aligned16(L) || !aligned16(A)) return FLAT_ERR_ALIGN;
    // (the row softmax runs one CTA per row of L: the row count is a grid dimension)
    if (static_cast<int64_t>(q.B) * q.H * q.Nq > 0x7fffffffLL) return FLAT_ERR_SHAPE;
    const int r = flat::launch_naive(q, L, A, static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 3;
    return r;
}

int flat_attn_naive_fwd(const void* Q, const void* K, const void* V, void* O, void* L, void* A, int B, int H,
                        int Nq, int Nk, int d, float scale, void* stream) {
    flat_attn_params_t p{Q, K, V, O, B, H, Nq, Nk, d, scale, FLAT_DTYPE_BF16, nullptr, nullptr, FLAT_VARIANT_AUTO, 0, nullptr, nullptr, 0, 0, 0, nullptr, 0, 0};
    return flat_attn_naive_fwd_ex(&p, L, A, stream);
}

int flat_attn_bwd_ex(const flat_attn_bwd_params_t* p, void* stream) {
    if (!p) return FLAT_ERR_NULL;
    if (!p->Q || !p->K || !p->V || !p->O || !p->dO || !p->lse || !p->dQ || !p->dK || !p->dV || !p->delta)
        return FLAT_ERR_NULL;
    // sizes, scale, masks and the alignment of Q, K, V, O: the forward's rules
    flat_attn_params_t f{p->Q, p->K, p->V, const_cast<void*>(p->O), p->B, p->H, p->Nq, p->Nk, p->d, p->scale,
                         FLAT_DTYPE_BF16, p->k_valid_len, p->status, FLAT_VARIANT_AUTO, p->causal, nullptr, nullptr, 0, 0, 0, nullptr, 0, 0};
    flat::Problem q;
    const int rc = validate(&f, &q);
    if (rc != FLAT_OK) return rc;
    if (p->d != 64 && p->d != 128) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(p->dO) || !aligned16(p->dQ) || !aligned16(p->dK) || !aligned16(p->dV)) return FLAT_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(p->lse) & 3u) || (reinterpret_cast<uintptr_t>(p->delta) & 3u)) return FLAT_ERR_ALIGN;
    const flat::BwdProblem b{p->Q, p->K, p->V, p->O, p->dO, p->lse, p->dQ, p->dK, p->dV, p->delta, p->B, p->H, p->Nq,
                             p->Nk, p->d, p->scale, p->k_valid_len, q.status, p->causal};
    const int r = flat::launch_bwd_tc(b, static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 2;
    return r;
}

int flat_attn_bwd(const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* lse,
                  void* dQ, void* dK, void* dV, float* delta, int B, int H, int Nq, int Nk, int d, float scale,
                  void* stream) {
    flat_attn_bwd_params_t p{Q, K, V, O, dO, lse, dQ, dK, dV, delta, B, H, Nq, Nk, d, scale, nullptr, nullptr, 0};
    return flat_attn_bwd_ex(&p, stream);
}

size_t flat_attn_host_workspace_bytes(int B, int H, int Nq, int Nk, int d, int dtype) {
    if (B < 1 || H < 1 || Nq < 1 || Nk < 1 || d < 1) return 0;
    const size_t es = dtype == FLAT_DTYPE_F32 ? 4 : 2;
    const size_t q = round256(es * B * H * static_cast<size_t>(Nq) * d);
    const size_t k = round256(es * B * H * static_cast<size_t>(Nk) * d);
    return 2 * q + 2 * k + round256(sizeof(int32_t) * static_cast<size_t>(B));
}

int flat_attn_fwd_host(const flat_attn_params_t* p, void* workspace, size_t workspace_bytes, void* stream) {
    if (!p || !workspace) return FLAT_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return FLAT_ERR_ALIGN;
    if (!p->Q || !p->K || !p->V || !p->O) return FLAT_ERR_NULL;
    if (p->B < 1 || p->H < 1 || p->Nq < 1 || p->Nk < 1 || p->d < 1) return FLAT_ERR_SHAPE;
    if (p->dtype != FLAT_DTYPE_BF16 && p->dtype != FLAT_DTYPE_F32) return FLAT_ERR_UNSUPPORTED;
    const size_t need = flat_attn_host_workspace_bytes(p->B, p->H, p->Nq, p->Nk, p->d, p->dtype);
    if (workspace_bytes < need) return FLAT_ERR_WORKSPACE;
    const size_t es = p->dtype == FLAT_DTYPE_F32 ? 4 : 2;
    const size_t qb = es * p->B * p->H * static_cast<size_t>(p->Nq) * p->d;
    const size_t kb = es * p->B * p->H * static_cast<size_t>(p->Nk) * p->d;
    char* w = static_cast<char*>(workspace);
    char* dQ = w;
    char* dK = dQ + round256(qb);
    char* dV = dK + round256(kb);
    char* dO = dV + round256(kb);
    char* dLen = dO + round256(qb);
    flat_attn_params_t dev = *p;
    dev.Q = dQ; dev.K = dK; dev.V = dV; dev.O = dO;
    dev.k_valid_len = p->k_valid_len ? reinterpret_cast<const int32_t*>(dLen) : nullptr;
    flat::Problem q;
    const int rc = validate(&dev, &q);
    if (rc != FLAT_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (p->k_valid_len &&
        cudaMemcpyAsync(dLen, p->k_valid_len, sizeof(int32_t) * p->B, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return FLAT_ERR_CUDA;

    // Pipeline over independent slices (whole batches, or groups of heads when B == 1): the copy of
    // slice c+1 overlaps the kernel of slice c and the read-back of slice c-1.  Two side streams
    // (created once per device; streams and events are not device memory) fork from `stream` and
    // join it again, so the caller sees ordinary stream semantics.
    HostPipe* hp = host_pipe();
    const int units = p->B > 1 ? p->B : p->H;            // slices are cut along this axis
    int nslices = units < 8 ? units : 8;
    if (!hp || nslices < 2) {
        if (cudaMemcpyAsync(dQ, p->Q, qb, cudaMemcpyHostToDevice, st) != cudaSuccess) return FLAT_ERR_CUDA;
        if (cudaMemcpyAsync(dK, p->K, kb, cudaMemcpyHostToDevice, st) != cudaSuccess) return FLAT_ERR_CUDA;
        if (cudaMemcpyAsync(dV, p->V, kb, cudaMemcpyHostToDevice, st) != cudaSuccess) return FLAT_ERR_CUDA;
        const int r = run_fused(q, p->variant, st);
        if (r != FLAT_OK) return r;
        if (cudaMemcpyAsync(p->O, dO, qb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FLAT_ERR_CUDA;
        g_last_launches = 1;
        return FLAT_OK;
    }
    if (cudaEventRecord(hp->fork, st) != cudaSuccess) return FLAT_ERR_CUDA;
    for (int i = 0; i < 2; ++i)
        if (cudaStreamWaitEvent(hp->side[i], hp->fork, 0) != cudaSuccess) return FLAT_ERR_CUDA;
    const size_t q_unit = qb / units, k_unit = kb / units;   // bytes per batch (or per head when B == 1)
    int launches = 0;
    for (int c = 0; c < nslices; ++c) {
        const int u0 = static_cast<int>(static_cast<int64_t>(units) * c / nslices);
        const int u1 = static_cast<int>(static_cast<int64_t>(units) * (c + 1) / nslices);
        if (u1 == u0) continue;
        cudaStream_t ss = hp->side[c & 1];
        const size_t qo = q_unit * u0, ko = k_unit * u0, qn = q_unit * (u1 - u0), kn = k_unit * (u1 - u0);
        if (cudaMemcpyAsync(dQ + qo, static_cast<const char*>(p->Q) + qo, qn, cudaMemcpyHostToDevice, ss) != cudaSuccess ||
            cudaMemcpyAsync(dK + ko, static_cast<const char*>(p->K) + ko, kn, cudaMemcpyHostToDevice, ss) != cudaSuccess ||
            cudaMemcpyAsync(dV + ko, static_cast<const char*>(p->V) + ko, kn, cudaMemcpyHostToDevice, ss) != cudaSuccess)
            return FLAT_ERR_CUDA;
        flat::Problem sub = q;
        sub.Q = dQ + qo; sub.K = dK + ko; sub.V = dV + ko; sub.O = dO + qo;
        if (p->B > 1) { sub.B = u1 - u0; if (sub.k_valid_len) sub.k_valid_len += u0; }
        else          { sub.H = u1 - u0; }
        if (sub.lse) sub.lse += static_cast<size_t>(u0) * (p->B > 1 ? static_cast<size_t>(p->H) * p->Nq : static_cast<size_t>(p->Nq));
        const int r = run_fused(sub, p->variant, ss);
        if (r != FLAT_OK) return r;
        ++launches;
        if (cudaMemcpyAsync(static_cast<char*>(p->O) + qo, dO + qo, qn, cudaMemcpyDeviceToHost, ss) != cudaSuccess)
            return FLAT_ERR_CUDA;
    }
    for (int i = 0; i < 2; ++i) {
        if (cudaEventRecord(hp->join[i], hp->side[i]) != cudaSuccess) return FLAT_ERR_CUDA;
        if (cudaStreamWaitEvent(st, hp->join[i], 0) != cudaSuccess) return FLAT_ERR_CUDA;
    }
    g_last_launches = launches;
    return FLAT_OK;
}

int flat_attn_selftest_exp2_poly(const float* x, float* y, int n, void* stream) {
    if (!x || !y) return FLAT_ERR_NULL;
    if (n < 1) return FLAT_ERR_SHAPE;
    const int r = flat::launch_exp2_poly_selftest(x, y, n, static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_attn_selftest_wait_timeout(int32_t* status, void* stream) {
    if (status && (reinterpret_cast<uintptr_t>(status) & 3u)) return FLAT_ERR_ALIGN;
    status = status_or_library_word(status);             // NULL: the code goes to the library's own word
    if (!status) return FLAT_ERR_CUDA;
    const int r = flat::launch_wait_timeout_selftest(status, static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_qkv_proj_fwd(const void* X, const void* Wqkv, void* Q, void* K, void* V, int B, int N, int H, int d,
                      int Dm, int32_t* status, void* stream) {
    const int r = flat::launch_qkv_proj(X, Wqkv, Q, K, V, B, N, H, d, Dm, status_or_library_word(status), static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_out_proj_fwd(const void* O, const void* Wo, void* Y, int B, int N, int H, int d, int Dm, int32_t* status,
                      void* stream) {
    const int r = flat::launch_out_proj(O, Wo, Y, B, N, H, d, Dm, status_or_library_word(status), static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_attn_varlen_fwd(const void* Q, const void* K, const void* V, void* O, const int32_t* cu_seqlens_q,
                         const int32_t* cu_seqlens_k, int num_seqs, int H, int d, long long total_q, long long total_k,
                         int max_seqlen_q, float scale, int causal, int32_t* status, void* stream) {
    if (!Q || !K || !V || !O || !cu_seqlens_q || !cu_seqlens_k) return FLAT_ERR_NULL;
    if (num_seqs < 1 || H < 1 || d < 1 || total_q < 1 || total_k < 1 || max_seqlen_q < 1 || !isfinite(scale))
        return FLAT_ERR_SHAPE;
    if (total_q > 0x7fffffffLL || total_k > 0x7fffffffLL || max_seqlen_q > total_q ||
        static_cast<int64_t>(num_seqs) * H > 0x7fffffffLL)
        return FLAT_ERR_SHAPE;
    if ((d != 64 && d != 128) || (causal != 0 && causal != 1)) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return FLAT_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(cu_seqlens_q) & 3u) || (reinterpret_cast<uintptr_t>(cu_seqlens_k) & 3u) ||
        (status && (reinterpret_cast<uintptr_t>(status) & 3u)))
        return FLAT_ERR_ALIGN;
    const int r = (d == 64 ? flat::launch_fused_tc3_varlen : flat::launch_fused_tc2_varlen)(
        Q, K, V, O, cu_seqlens_q, cu_seqlens_k, num_seqs, H, total_q, total_k, max_seqlen_q, scale, causal,
        status_or_library_word(status),
        static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_fc_fwd(const void* X, const void* W, void* Y, int M, int K, int Nout, int32_t* status, void* stream) {
    const int r = flat::launch_fc(X, W, Y, M, K, Nout, status_or_library_word(status), static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_layernorm_fwd(const void* X, const void* R, const void* gamma, const void* beta, void* Y, long long M, int D,
                       float eps, void* stream) {
    if (!X || !gamma || !beta || !Y) return FLAT_ERR_NULL;
    if (M < 1 || D < 1 || !(eps >= 0.f) || !isfinite(eps)) return FLAT_ERR_SHAPE;
    if (M > INT64_MAX / 16 / D) return FLAT_ERR_SHAPE;
    if (D % 8 != 0 || D > 8192) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(gamma) || !aligned16(beta) || !aligned16(Y) || (R && !aligned16(R))) return FLAT_ERR_ALIGN;
    const int r = flat::launch_layernorm(X, R, gamma, beta, Y, M, D, eps, static_cast<cudaStream_t>(stream));
    if (r == FLAT_OK) g_last_launches = 1;
    return r;
}

int flat_attn_layer_fwd(const void* X, const void* Wqkv, const void* Wo, void* Y, void* Q, void* K, void* V, void* O,
                        int B, int N, int H, int d, int Dm, float scale, int causal, int32_t* status, void* stream) {
    if (!X || !Wqkv || !Wo || !Y || !Q || !K || !V || !O) return FLAT_ERR_NULL;
    // validate all three steps before anything is launched
    flat_attn_params_t p{Q, K, V, O, B, H, N, N, d, scale, FLAT_DTYPE_BF16, nullptr, status, FLAT_VARIANT_AUTO, causal, nullptr, nullptr, 0, 0, 0, nullptr, 0, 0};
    flat::Problem q;
    int rc = validate(&p, &q);
    if (rc != FLAT_OK) return rc;
    if ((d != 64 && d != 128) || (H * d) % 256 != 0 || Dm % 256 != 0 || N % 128 != 0) return FLAT_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(Wqkv) || !aligned16(Wo) || !aligned16(Y)) return FLAT_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = flat::launch_qkv_proj(X, Wqkv, Q, K, V, B, N, H, d, Dm, status_or_library_word(status), st);
    if (rc != FLAT_OK) return rc;
    rc = run_fused(q, FLAT_VARIANT_AUTO, st);
    if (rc != FLAT_OK) return rc;
    rc = flat::launch_out_proj(O, Wo, Y, B, N, H, d, Dm, status_or_library_word(status), st);
    if (rc == FLAT_OK) g_last_launches = 3;
    return rc;
}

int flat_attn_last_launch_count(void) { return g_last_launches; }

int flat_attn_last_variant(void) { return g_last_variant; }

int flat_attn_last_schedule(void) { return flat::g_last_schedule; }

int flat_attn_last_device_error(int32_t* code) {
    if (!code) return FLAT_ERR_NULL;
    int32_t* w = library_status_word();
    if (!w) return FLAT_ERR_CUDA;
    return cudaMemcpy(code, w, sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

int flat_attn_clear_device_error(void) {
    int32_t* w = library_status_word();
    if (!w) return FLAT_ERR_CUDA;
    return cudaMemset(w, 0, sizeof(int32_t)) == cudaSuccess ? FLAT_OK : FLAT_ERR_CUDA;
}

const char* flat_attn_status_string(int code) {
    switch (code) {
        case FLAT_OK: return "ok";
        case FLAT_ERR_NULL: return "required pointer is NULL";
        case FLAT_ERR_SHAPE: return "bad size or scale";
        case FLAT_ERR_UNSUPPORTED: return "unsupported d, dtype or variant";
        case FLAT_ERR_ALIGN: return "pointer not aligned";
        case FLAT_ERR_WORKSPACE: return "workspace too small";
        case FLAT_ERR_CUDA: return "CUDA call failed";
        case FLAT_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int flat_attn_version(void) { return 100; }

}  // extern "C"

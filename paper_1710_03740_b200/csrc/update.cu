// Master-weight pass (paper sections 3.1, 3.2): recast, overflow inspection, and the
// fused unscale / inspect / FP32 SGD(+momentum) / FP16 re-round kernel.
//
// All three are streaming kernels bound by HBM bandwidth: 64- and 128-bit accesses with streaming
// cache hints, one CTA of 256 threads per 8192 consecutive parameters (320 bytes of loads in
// flight per thread, all issued before the first use) and no grid-stride loop: on B200 a grid of short-lived CTAs handed out in address order by the
// hardware scheduler sustains about 20 % more bandwidth than a persistent grid-stride grid.
// The update reads g16, w32, (v) once and writes w32, (v), w16 once: 12 bytes/parameter
// (plain SGD) or 20 bytes/parameter (momentum).
//
// Bit-exactness contract: every FP32 operation is rounded separately (the __f*_rn
// intrinsics are never contracted into a fused multiply-add), no flush-to-zero.
#include "mpt_common.cuh"
#include "update_math.cuh"

namespace mpt {

static constexpr int kThreads = 256;
static constexpr int kSMs = 148;
static constexpr int kCtasPerSM = 8;
static constexpr int kVecPerThread = 4;   // 8-element vectors per thread in the one-shot kernels
static constexpr int kUnitsPerThread = 8; // 4-element units per thread in the master pass

__device__ __forceinline__ float h2f_bits(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }
__device__ __forceinline__ uint32_t f2h_bits(float x) { return (uint32_t)__half_as_ushort(__float2half_rn(x)); }

static inline int grid_for(size_t work_items)
{
    size_t blocks = (work_items + kThreads - 1) / kThreads;
    size_t cap = (size_t)kSMs * kCtasPerSM;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// one CTA per kThreads * kVecPerThread vectors
static inline unsigned vec_grid(size_t n8)
{
    const size_t per_cta = (size_t)kThreads * kVecPerThread;
    return (unsigned)((n8 + per_cta - 1) / per_cta);
}

// ------------------------------------------------------------------ recast

__global__ void __launch_bounds__(kThreads) k_recast_vec(const float4 *__restrict__ w32, uint4 *__restrict__ w16,
                                                         size_t n8)
{
    pdl_trigger();
    pdl_wait();
    const size_t base = (size_t)blockIdx.x * (kThreads * kVecPerThread) + threadIdx.x;
    float4 a[kVecPerThread], b[kVecPerThread];
#pragma unroll
    for (int u = 0; u < kVecPerThread; u++) {
        const size_t j = base + (size_t)u * kThreads;
        if (j < n8) { a[u] = __ldcs(w32 + 2 * j); b[u] = __ldcs(w32 + 2 * j + 1); }
    }
#pragma unroll
    for (int u = 0; u < kVecPerThread; u++) {
        const size_t j = base + (size_t)u * kThreads;
        if (j < n8) {
            uint4 o;
            o.x = f2h_bits(a[u].x) | (f2h_bits(a[u].y) << 16);
            o.y = f2h_bits(a[u].z) | (f2h_bits(a[u].w) << 16);
            o.z = f2h_bits(b[u].x) | (f2h_bits(b[u].y) << 16);
            o.w = f2h_bits(b[u].z) | (f2h_bits(b[u].w) << 16);
            w16[j] = o;
        }
    }
}

__global__ void k_recast_scalar(const float *__restrict__ w32, uint16_t *__restrict__ w16, size_t begin, size_t n)
{
    pdl_trigger();
    pdl_wait();
    size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        w16[i] = (uint16_t)f2h_bits(w32[i]);
}

cudaError_t launch_recast(const float *w32, uint16_t *w16, size_t n, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    bool aligned = (((uintptr_t)w32 | (uintptr_t)w16) & 15) == 0;
    size_t n8 = aligned ? n / 8 : 0;
    if (n8) MPT_LAUNCH(k_recast_vec, dim3(vec_grid(n8)), dim3(kThreads), 0, st, (const float4 *)w32, (uint4 *)w16, n8);
    if (n8 * 8 < n) MPT_LAUNCH(k_recast_scalar, dim3(grid_for(n - n8 * 8)), dim3(kThreads), 0, st, w32, w16, n8 * 8, n);
    return cudaGetLastError();
}

// ------------------------------------------------------- overflow inspection

__device__ __forceinline__ bool pair_nonfinite(uint32_t two_halfs, float inv)
{
    return f32_nonfinite(__fmul_rn(h2f_bits(two_halfs & 0xFFFFu), inv)) ||
           f32_nonfinite(__fmul_rn(h2f_bits(two_halfs >> 16), inv));
}

__global__ void __launch_bounds__(kThreads) k_nonfinite_vec(const uint4 *__restrict__ g, size_t n8, float inv,
                                                            uint32_t *flag)
{
    pdl_trigger();
    pdl_wait();
    const size_t base = (size_t)blockIdx.x * (kThreads * kVecPerThread) + threadIdx.x;
    uint4 x[kVecPerThread];
#pragma unroll
    for (int u = 0; u < kVecPerThread; u++) {
        const size_t j = base + (size_t)u * kThreads;
        x[u] = (j < n8) ? __ldcs(g + j) : make_uint4(0, 0, 0, 0);
    }
    bool bad = false;
#pragma unroll
    for (int u = 0; u < kVecPerThread; u++)
        bad |= pair_nonfinite(x[u].x, inv) | pair_nonfinite(x[u].y, inv) | pair_nonfinite(x[u].z, inv) |
               pair_nonfinite(x[u].w, inv);
    // warp vote, then at most one atomic per warp and only when something was found
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flag, 1u);
}

__global__ void k_nonfinite_scalar(const uint16_t *__restrict__ g, size_t begin, size_t n, float inv, uint32_t *flag)
{
    pdl_trigger();
    pdl_wait();
    size_t stride = (size_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (size_t i = begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        bad |= f32_nonfinite(__fmul_rn(h2f_bits(g[i]), inv));
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flag, 1u);
}

cudaError_t launch_grad_nonfinite(const uint16_t *g16, size_t n, float inv_S, uint32_t *flag, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    bool aligned = ((uintptr_t)g16 & 15) == 0;
    size_t n8 = aligned ? n / 8 : 0;
    if (n8) MPT_LAUNCH(k_nonfinite_vec, dim3(vec_grid(n8)), dim3(kThreads), 0, st, (const uint4 *)g16, n8, inv_S, flag);
    if (n8 * 8 < n) MPT_LAUNCH(k_nonfinite_scalar, dim3(grid_for(n - n8 * 8)), dim3(kThreads), 0, st, g16, n8 * 8, n, inv_S, flag);
    return cudaGetLastError();
}

// ------------------------------------------------------------------- update

// One element: g = f32(g16) * inv ; [v = mu*v + g ; u = lr*v] or [u = lr*g] ; w -= u.
template <bool MOM>
__device__ __forceinline__ void upd1(uint32_t gh, float &w, float &v, float inv, float lr, float mu, bool &bad)
{
    float g = __fmul_rn(h2f_bits(gh), inv);
    bad |= f32_nonfinite(g);
    float u;
    if (MOM) {
        float t = __fmul_rn(mu, v);
        v = __fadd_rn(t, g);
        u = __fmul_rn(lr, v);
    } else {
        u = __fmul_rn(lr, g);
    }
    w = __fsub_rn(w, u);
}

template <bool MOM>
__device__ __forceinline__ void upd8(const uint4 &g, float4 &w0, float4 &w1, float4 &v0, float4 &v1, uint4 &h,
                                     float inv, float lr, float mu, bool &bad)
{
    upd1<MOM>(g.x & 0xFFFFu, w0.x, v0.x, inv, lr, mu, bad);
    upd1<MOM>(g.x >> 16, w0.y, v0.y, inv, lr, mu, bad);
    upd1<MOM>(g.y & 0xFFFFu, w0.z, v0.z, inv, lr, mu, bad);
    upd1<MOM>(g.y >> 16, w0.w, v0.w, inv, lr, mu, bad);
    upd1<MOM>(g.z & 0xFFFFu, w1.x, v1.x, inv, lr, mu, bad);
    upd1<MOM>(g.z >> 16, w1.y, v1.y, inv, lr, mu, bad);
    upd1<MOM>(g.w & 0xFFFFu, w1.z, v1.z, inv, lr, mu, bad);
    upd1<MOM>(g.w >> 16, w1.w, v1.w, inv, lr, mu, bad);
    h.x = f2h_bits(w0.x) | (f2h_bits(w0.y) << 16);
    h.y = f2h_bits(w0.z) | (f2h_bits(w0.w) << 16);
    h.z = f2h_bits(w1.x) | (f2h_bits(w1.y) << 16);
    h.w = f2h_bits(w1.z) | (f2h_bits(w1.w) << 16);
}

// flags[0]: overflow decided by the producer of the gradients (read, never written);
// flags[1]: this kernel's own inspection (written).  When flags[0] is set the whole
// grid returns before touching a parameter: a skipped step moves no parameter byte.
// Work unit: 4 consecutive parameters.  Every thread reads 8 bytes of gradients and 16 + 16 bytes
// of master and momentum per unit, so each warp-wide access covers whole, consecutive 32-byte
// sectors exactly once.  (With 8-parameter units a thread reads its two float4 halves of w32 with
// a 32-byte stride between neighbouring lanes: twice the sector requests per instruction.  That
// form was level at full clock but 13 % slower at the 1.3 GHz the SMs run at right after the
// power-capped products of a training step - 5.52 against 4.78 ms for 1.6 G parameters there.)
// UPT units per thread, all loads issued before the first use.
template <bool MOM, int UPT>
__global__ void __launch_bounds__(kThreads) k_update_quad(const uint2 *__restrict__ g16, float4 *__restrict__ w32,
                                                          float4 *__restrict__ v32, uint2 *__restrict__ w16, size_t n4,
                                                          float inv, float lr, float mu, uint32_t *flags,
                                                          const float *__restrict__ inv_dev)
{
    pdl_trigger();
    pdl_wait();
    if (*(volatile const uint32_t *)flags != 0u) return;
    if (inv_dev) inv = *inv_dev;
    const size_t base = (size_t)blockIdx.x * (kThreads * UPT) + threadIdx.x;
    bool bad = false;
    uint2 g[UPT];
    float4 w[UPT], v[UPT];
#pragma unroll
    for (int u = 0; u < UPT; u++) {
        const size_t j = base + (size_t)u * kThreads;
        if (j < n4) {
            g[u] = __ldcs(g16 + j);
            w[u] = __ldcs(w32 + j);
            if (MOM) v[u] = __ldcs(v32 + j);
        }
    }
#pragma unroll
    for (int u = 0; u < UPT; u++) {
        const size_t j = base + (size_t)u * kThreads;
        if (j < n4) {
            if (!MOM) v[u] = make_float4(0, 0, 0, 0);
            upd1<MOM>(g[u].x & 0xFFFFu, w[u].x, v[u].x, inv, lr, mu, bad);
            upd1<MOM>(g[u].x >> 16, w[u].y, v[u].y, inv, lr, mu, bad);
            upd1<MOM>(g[u].y & 0xFFFFu, w[u].z, v[u].z, inv, lr, mu, bad);
            upd1<MOM>(g[u].y >> 16, w[u].w, v[u].w, inv, lr, mu, bad);
            uint2 h;
            h.x = f2h_bits(w[u].x) | (f2h_bits(w[u].y) << 16);
            h.y = f2h_bits(w[u].z) | (f2h_bits(w[u].w) << 16);
            __stcs(w32 + j, w[u]);
            if (MOM) __stcs(v32 + j, v[u]);
            __stcs(w16 + j, h);
        }
    }
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flags + 1, 1u);
}

template <bool MOM>
__global__ void k_update_scalar(const uint16_t *__restrict__ g16, float *__restrict__ w32, float *__restrict__ v32,
                                uint16_t *__restrict__ w16, size_t begin, size_t n, float inv, float lr, float mu,
                                uint32_t *flags, const float *__restrict__ inv_dev)
{
    pdl_trigger();
    pdl_wait();
    if (*(volatile const uint32_t *)flags != 0u) return;
    if (inv_dev) inv = *inv_dev;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (size_t i = begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float w = w32[i], v = MOM ? v32[i] : 0.0f;
        upd1<MOM>(g16[i], w, v, inv, lr, mu, bad);
        w32[i] = w;
        if (MOM) v32[i] = v;
        w16[i] = (uint16_t)f2h_bits(w);
    }
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flags + 1, 1u);
}

cudaError_t launch_update(const uint16_t *g16, float *w32, float *v, uint16_t *w16, size_t n, float inv_S, float lr,
                          float mu, bool use_momentum, uint32_t *flags, cudaStream_t st, const float *inv_S_dev)
{
    if (n == 0) return cudaSuccess;
    uintptr_t bits = (uintptr_t)g16 | (uintptr_t)w32 | (uintptr_t)w16 | (use_momentum ? (uintptr_t)v : 0);
    size_t n8 = (bits & 15) == 0 ? n / 8 : 0;
    if (n8) {
        const size_t n4 = n8 * 2;
        const unsigned grid = (unsigned)((n4 + (size_t)kThreads * kUnitsPerThread - 1) / ((size_t)kThreads * kUnitsPerThread));
        if (use_momentum)
            MPT_LAUNCH((k_update_quad<true, kUnitsPerThread>), dim3(grid), dim3(kThreads), 0, st, (const uint2 *)g16, (float4 *)w32,
                       (float4 *)v, (uint2 *)w16, n4, inv_S, lr, mu, flags, inv_S_dev);
        else
            MPT_LAUNCH((k_update_quad<false, kUnitsPerThread>), dim3(grid), dim3(kThreads), 0, st, (const uint2 *)g16, (float4 *)w32,
                       nullptr, (uint2 *)w16, n4, inv_S, lr, mu, flags, inv_S_dev);
    }
    if (n8 * 8 < n) {
        int grid = grid_for(n - n8 * 8);
        if (use_momentum)
            MPT_LAUNCH(k_update_scalar<true>, dim3(grid), dim3(kThreads), 0, st, g16, w32, v, w16, n8 * 8, n, inv_S, lr, mu, flags, inv_S_dev);
        else
            MPT_LAUNCH(k_update_scalar<false>, dim3(grid), dim3(kThreads), 0, st, g16, w32, nullptr, w16, n8 * 8, n, inv_S, lr, mu, flags, inv_S_dev);
    }
    return cudaGetLastError();
}

// ------------------------------------------- other optimizer steps, weight decay

static constexpr int kOptUnits = 4;   // 4-element units per thread (up to 56 bytes of loads each)

// Same structure as k_update_quad: units of 4 consecutive parameters, whole sectors per warp access.
template <int KIND, bool WD>
__global__ void __launch_bounds__(kThreads) k_update_opt(const uint2 *__restrict__ g16, float4 *__restrict__ w32,
                                                         float4 *__restrict__ s1p, float4 *__restrict__ s2p,
                                                         uint2 *__restrict__ w16, size_t n4, float inv, float lr, float mu,
                                                         float b2, float eps, float wd, float b1t, float b2t,
                                                         uint32_t *flags, const float *__restrict__ inv_dev,
                                                         const float *__restrict__ betat_dev,
                                                         const float *__restrict__ coef_dev)
{
    pdl_trigger();
    pdl_wait();
    if (*(volatile const uint32_t *)flags != 0u) return;
    if (inv_dev) inv = *inv_dev;
    const float coef = coef_dev ? *coef_dev : 1.0f;
    if (betat_dev) { b1t = __fmul_rn(betat_dev[0], mu); b2t = __fmul_rn(betat_dev[1], b2); }
    const float bc1 = __fsub_rn(1.0f, b1t), bc2 = __fsub_rn(1.0f, b2t);
    const float omb1 = __fsub_rn(1.0f, mu), omb2 = __fsub_rn(1.0f, b2);
    constexpr bool S2 = KIND == MPT_OPT_ADAM;
    const bool use_s1 = KIND != MPT_OPT_SGD || mu != 0.0f;      // every kind handled here may use the first state
    const size_t base = (size_t)blockIdx.x * (kThreads * kOptUnits) + threadIdx.x;
    bool bad = false;
    uint2 g[kOptUnits];
    float4 w[kOptUnits], a[kOptUnits], b[kOptUnits];
#pragma unroll
    for (int u = 0; u < kOptUnits; u++) {
        const size_t j = base + (size_t)u * kThreads;
        a[u] = b[u] = make_float4(0, 0, 0, 0);
        if (j < n4) {
            g[u] = __ldcs(g16 + j);
            w[u] = __ldcs(w32 + j);
            if (use_s1) a[u] = __ldcs(s1p + j);
            if (S2) b[u] = __ldcs(s2p + j);
        }
    }
#pragma unroll
    for (int u = 0; u < kOptUnits; u++) {
        const size_t j = base + (size_t)u * kThreads;
        if (j < n4) {
            const uint32_t gw[2] = {g[u].x, g[u].y};
            float *wf = &w[u].x, *af = &a[u].x, *bf = &b[u].x;
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const uint32_t gh = (e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu);
                opt1<KIND, WD>(h2f_bits(gh), wf[e], af[e], bf[e], inv, lr, mu, b2, omb1, omb2, eps, wd, bc1, bc2, coef, bad);
            }
            uint2 h;
            h.x = f2h_bits(w[u].x) | (f2h_bits(w[u].y) << 16);
            h.y = f2h_bits(w[u].z) | (f2h_bits(w[u].w) << 16);
            __stcs(w32 + j, w[u]);
            if (use_s1) __stcs(s1p + j, a[u]);
            if (S2) __stcs(s2p + j, b[u]);
            __stcs(w16 + j, h);
        }
    }
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flags + 1, 1u);
}

template <int KIND, bool WD>
__global__ void k_update_opt_scalar(const uint16_t *__restrict__ g16, float *__restrict__ w32, float *__restrict__ s1p,
                                    float *__restrict__ s2p, uint16_t *__restrict__ w16, size_t begin, size_t n, float inv,
                                    float lr, float mu, float b2, float eps, float wd, float b1t, float b2t, uint32_t *flags,
                                    const float *__restrict__ inv_dev, const float *__restrict__ betat_dev,
                                    const float *__restrict__ coef_dev)
{
    pdl_trigger();
    pdl_wait();
    if (*(volatile const uint32_t *)flags != 0u) return;
    if (inv_dev) inv = *inv_dev;
    const float coef = coef_dev ? *coef_dev : 1.0f;
    if (betat_dev) { b1t = __fmul_rn(betat_dev[0], mu); b2t = __fmul_rn(betat_dev[1], b2); }
    const float bc1 = __fsub_rn(1.0f, b1t), bc2 = __fsub_rn(1.0f, b2t);
    const float omb1 = __fsub_rn(1.0f, mu), omb2 = __fsub_rn(1.0f, b2);
    const bool use_s1 = KIND != MPT_OPT_SGD || mu != 0.0f;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (size_t i = begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        float w = w32[i], a = use_s1 ? s1p[i] : 0.0f, b = KIND == MPT_OPT_ADAM ? s2p[i] : 0.0f;
        opt1<KIND, WD>(h2f_bits(g16[i]), w, a, b, inv, lr, mu, b2, omb1, omb2, eps, wd, bc1, bc2, coef, bad);
        w32[i] = w;
        if (use_s1) s1p[i] = a;
        if (KIND == MPT_OPT_ADAM) s2p[i] = b;
        w16[i] = (uint16_t)f2h_bits(w);
    }
    if (__any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(flags + 1, 1u);
}

template <int KIND, bool WD>
static cudaError_t launch_opt_variant(const uint16_t *g16, float *w32, float *s1, float *s2, uint16_t *w16, size_t n,
                                      float inv_S, float lr, float mu, float b2, float eps, float wd, float b1t, float b2t,
                                      uint32_t *flags, cudaStream_t st, const float *inv_dev, const float *betat_dev,
                                      const float *coef_dev)
{
    uintptr_t bits = (uintptr_t)g16 | (uintptr_t)w32 | (uintptr_t)w16 | (uintptr_t)s1 | (uintptr_t)s2;
    size_t n8 = (bits & 15) == 0 ? n / 8 : 0;
    if (n8) {
        const size_t n4 = n8 * 2, per_cta = (size_t)kThreads * kOptUnits;
        MPT_LAUNCH((k_update_opt<KIND, WD>), dim3((unsigned)((n4 + per_cta - 1) / per_cta)), dim3(kThreads), 0, st,
                   (const uint2 *)g16, (float4 *)w32, (float4 *)s1, (float4 *)s2, (uint2 *)w16, n4, inv_S, lr, mu, b2, eps, wd, b1t, b2t,
                   flags, inv_dev, betat_dev, coef_dev);
    }
    if (n8 * 8 < n)
        MPT_LAUNCH(k_update_opt_scalar<KIND, WD>, dim3(grid_for(n - n8 * 8)), dim3(kThreads), 0, st, g16, w32, s1, s2, w16, n8 * 8, n, inv_S, lr, mu, b2,
                   eps, wd, b1t, b2t, flags, inv_dev, betat_dev, coef_dev);
    return cudaGetLastError();
}

cudaError_t launch_update_opt(int kind, const uint16_t *g16, float *w32, float *s1, float *s2, uint16_t *w16, size_t n,
                              float inv_S, float lr, float mu, float b2, float eps, float wd, float b1t, float b2t,
                              uint32_t *flags, cudaStream_t st, const float *inv_dev, const float *betat_dev,
                              const float *coef_dev)
{
    if (n == 0) return cudaSuccess;
#define MPT_OPT_CASE(K)                                                                                                     \
    case K:                                                                                                                 \
        return wd != 0.0f ? launch_opt_variant<K, true>(g16, w32, s1, s2, w16, n, inv_S, lr, mu, b2, eps, wd, b1t, b2t, flags, \
                                                        st, inv_dev, betat_dev, coef_dev)                                   \
                          : launch_opt_variant<K, false>(g16, w32, s1, s2, w16, n, inv_S, lr, mu, b2, eps, wd, b1t, b2t, flags, \
                                                         st, inv_dev, betat_dev, coef_dev);
    switch (kind) {
        MPT_OPT_CASE(MPT_OPT_SGD)
        MPT_OPT_CASE(MPT_OPT_NESTEROV)
        MPT_OPT_CASE(MPT_OPT_ADAGRAD)
        MPT_OPT_CASE(MPT_OPT_ADAM)
        default: return cudaErrorInvalidValue;
    }
#undef MPT_OPT_CASE
}

__global__ void k_post_step(uint32_t *status, int interval, float backoff, float growth, float min_S, float max_S, int adam,
                            float b1, float b2)
{
    pdl_trigger();
    pdl_wait();
    const bool overflow = status[ST_OVERFLOW] != 0u;
    if (adam && !overflow) {
        status[ST_B1T] = __float_as_uint(__fmul_rn(__uint_as_float(status[ST_B1T]), b1));
        status[ST_B2T] = __float_as_uint(__fmul_rn(__uint_as_float(status[ST_B2T]), b2));
    }
    if (interval > 0) {
        float S = __uint_as_float(status[ST_SCALE]);
        uint32_t clean = status[ST_CLEAN_STEPS];
        if (overflow) {
            S = fmaxf(__fmul_rn(S, backoff), min_S);
            clean = 0;
        } else if (++clean >= (uint32_t)interval) {
            S = fminf(__fmul_rn(S, growth), max_S);
            clean = 0;
        }
        status[ST_SCALE] = __float_as_uint(S);
        status[ST_INV_SCALE] = __float_as_uint(__fdiv_rn(1.0f, S));
        status[ST_CLEAN_STEPS] = clean;
    }
}

cudaError_t launch_post_step(uint32_t *status, int interval, float backoff, float growth, float min_S, float max_S, int adam,
                             float b1, float b2, cudaStream_t st)
{
    MPT_LAUNCH(k_post_step, dim3(1), dim3(1), 0, st, status, interval, backoff, growth, min_S, max_S, adam, b1, b2);
    return cudaGetLastError();
}

// ------------------------------------------------------- dynamic loss scale

// The paper's closing section proposes raising or lowering the scale by inspecting the weight
// gradients for overflow while skipping the overflowing updates; it gives no schedule.  Taken
// here: multiply by `backoff` on overflow, by `growth` after `interval` clean steps in a row,
// clamp to [min_S, max_S].  With power-of-two factors every scale stays a power of two.
__global__ void k_scale_adjust(uint32_t *status, int interval, float backoff, float growth, float min_S, float max_S)
{
    pdl_trigger();
    pdl_wait();
    float S = __uint_as_float(status[ST_SCALE]);
    uint32_t clean = status[ST_CLEAN_STEPS];
    if (status[ST_OVERFLOW] != 0u) {
        S = fmaxf(__fmul_rn(S, backoff), min_S);
        clean = 0;
    } else if (++clean >= (uint32_t)interval) {
        S = fminf(__fmul_rn(S, growth), max_S);
        clean = 0;
    }
    status[ST_SCALE] = __float_as_uint(S);
    status[ST_INV_SCALE] = __float_as_uint(__fdiv_rn(1.0f, S));
    status[ST_CLEAN_STEPS] = clean;
}

cudaError_t launch_scale_adjust(uint32_t *status, int interval, float backoff, float growth, float min_S, float max_S,
                                cudaStream_t st)
{
    MPT_LAUNCH(k_scale_adjust, dim3(1), dim3(1), 0, st, status, interval, backoff, growth, min_S, max_S);
    return cudaGetLastError();
}

// ------------------------------------------------- global-norm gradient clipping

// Section 3.2: clipping thresholds act on the UNSCALED gradients.  The squared norm is accumulated
// in double (section 3.3: reductions in higher precision than the stored values) with a fixed
// partition, so the same input gives the same bits on every run: thread t of CTA b sums the
// vectors b*kThreads + t + k*kNormParts*kThreads in increasing k, a CTA combines its threads with
// a fixed shuffle/shared tree into parts[b], and one CTA combines the parts the same way.
__device__ __forceinline__ double block_sum_fixed(double v, double *sh)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if ((threadIdx.x & 31) == 0) sh[warp] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < nwarps; w++) total += sh[w];
    return total;   // valid in thread 0
}

__global__ void __launch_bounds__(kThreads) k_grad_sqnorm(const uint16_t *__restrict__ g16, size_t n, size_t n8, float inv,
                                                          const float *__restrict__ inv_dev, double *__restrict__ parts)
{
    pdl_trigger();
    pdl_wait();
    __shared__ double sh[kThreads / 32];
    if (inv_dev) inv = *inv_dev;
    double acc = 0.0;
    const uint4 *gv = (const uint4 *)g16;
    const size_t stride = (size_t)gridDim.x * kThreads;
    for (size_t j = (size_t)blockIdx.x * kThreads + threadIdx.x; j < n8; j += stride) {
        const uint4 q = __ldcs(gv + j);
        const uint32_t gw[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 8; e++) {
            const uint32_t gh = (e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu);
            const double v = (double)__fmul_rn(h2f_bits(gh), inv);
            acc += v * v;
        }
    }
    if (blockIdx.x == 0)      // elements past the last whole vector (or everything, for unaligned input)
        for (size_t i = n8 * 8 + threadIdx.x; i < n; i += kThreads) {
            const double v = (double)__fmul_rn(h2f_bits(g16[i]), inv);
            acc += v * v;
        }
    const double total = block_sum_fixed(acc, sh);
    if (threadIdx.x == 0) parts[blockIdx.x] = total;
}

// coef = min(1, clip / (sqrt(total) + 1e-6)) rounded to FP32; out[0] = coef, out[1] = norm (FP32).
__global__ void __launch_bounds__(1024) k_clip_coef(const double *__restrict__ parts, int count, float clip,
                                                    float *__restrict__ out)
{
    pdl_trigger();
    pdl_wait();
    __shared__ double sh[32];
    double acc = 0.0;
    for (int i = threadIdx.x; i < count; i += 1024) acc += parts[i];
    const double total = block_sum_fixed(acc, sh);
    if (threadIdx.x == 0) {
        const double norm = sqrt(total);
        out[0] = (float)fmin(1.0, (double)clip / (norm + 1e-6));
        out[1] = (float)norm;
    }
}

cudaError_t launch_clip_coef(const uint16_t *g16, size_t n, float inv_S, const float *inv_dev, float clip, double *parts,
                             float *out2, cudaStream_t st)
{
    const size_t n8 = ((uintptr_t)g16 & 15) == 0 ? n / 8 : 0;
    size_t want = (n8 + kThreads - 1) / kThreads;
    const int grid = (int)(want < 1 ? 1 : (want > (size_t)kNormParts ? (size_t)kNormParts : want));
    MPT_LAUNCH(k_grad_sqnorm, dim3(grid), dim3(kThreads), 0, st, g16, n, n8, inv_S, inv_dev, parts);
    MPT_LAUNCH(k_clip_coef, dim3(1), dim3(1024), 0, st, parts, grid, clip, out2);
    return cudaGetLastError();
}

}  // namespace mpt

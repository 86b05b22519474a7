// Data-parallel step (the paper's language model aggregates its batch over 4 GPUs, section 4.5):
// gradient exchange, master-weight pass and weight broadcast for one replica's shard of the
// parameters in ONE kernel over peer memory.  The owner of a shard pulls that shard of every
// replica's FP16 gradient (each element crosses the link once), adds them in FP32 in replica order,
// applies the update of sections 3.1 / 3.2 to its FP32 master shard, and pushes the re-rounded FP16
// weights into every replica's working copy.  Plain loads and stores on peer pointers only: no
// waits on other replicas inside the kernel (the caller orders the replicas around the call), no
// multicast.  Arithmetic contract: include/mpt.h (mpt_dp_step_flat).  k_dp_reduce is the first half (pull
// and sum) by itself, for running it layer by layer beside the backward pass; the step kernels then take
// the sums in place of the gradients.
#include <string.h>

#include "mpt_common.cuh"
#include "update_math.cuh"

namespace mpt {

namespace {

constexpr int kDpThreads = 256;

struct DpPeers {
    const uint16_t *g[MPT_DP_MAX_REPLICAS];
    const uint32_t *flag[MPT_DP_MAX_REPLICAS];
    uint16_t *w[MPT_DP_MAX_REPLICAS];
};

__device__ __forceinline__ float h2f_bits_dp(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }
__device__ __forceinline__ uint32_t f2h_bits_dp(float x) { return (uint32_t)__half_as_ushort(__float2half_rn(x)); }

// one element: s is the FP32 sum of the replicas' scaled gradients
template <bool MOM>
__device__ __forceinline__ void dp_elem(float s, float inv, float lr, float mu, float &w, float &v, bool &bad)
{
    const float g = __fmul_rn(s, inv);
    bad |= f32_nonfinite(g);
    float u;
    if (MOM) {
        v = __fadd_rn(__fmul_rn(mu, v), g);
        u = __fmul_rn(lr, v);
    } else {
        u = __fmul_rn(lr, g);
    }
    w = __fsub_rn(w, u);
}

__device__ __forceinline__ bool any_replica_overflowed(const DpPeers &pp, int R)
{
    uint32_t any = 0;
    for (int q = 0; q < R; q++) any |= *(volatile const uint32_t *)pp.flag[q];
    return any != 0;
}

// RT: replica count known at compile time (the loads of all replicas are then issued before the
// first addition), 0: any count.  `first` is the index of the shard's first element in the
// replicas' full-length arrays; w32 / v point at that element of the owner's state.
template <int RT, bool MOM>
__global__ void __launch_bounds__(kDpThreads) k_dp_step(const DpPeers pp, int R_dyn, float4 *__restrict__ w32,
                                                        float4 *__restrict__ v, size_t first, size_t n8, float inv,
                                                        const float *__restrict__ S_dev, float lr, float mu,
                                                        uint32_t *flags)
{
    pdl_trigger();
    pdl_wait();
    const int R = RT ? RT : R_dyn;
    if (S_dev) inv = __fdiv_rn(1.0f, __fmul_rn(*S_dev, (float)R));
    if (any_replica_overflowed(pp, R)) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(flags, 1u);
        return;
    }
    const size_t j = (size_t)blockIdx.x * kDpThreads + threadIdx.x;
    if (j >= n8) return;
    const size_t vec = first / 8 + j;          // `first` is a multiple of 8
    float s[8];
    if (RT) {
        uint4 g[RT ? RT : 1];
#pragma unroll
        for (int q = 0; q < RT; q++) g[q] = __ldcs((const uint4 *)pp.g[q] + vec);
#pragma unroll
        for (int q = 0; q < RT; q++) {
            const uint32_t gw[4] = {g[q].x, g[q].y, g[q].z, g[q].w};
#pragma unroll
            for (int e = 0; e < 8; e++) {
                const float x = h2f_bits_dp((e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu));
                s[e] = q == 0 ? x : __fadd_rn(s[e], x);
            }
        }
    } else {
        for (int q = 0; q < R; q++) {
            const uint4 g = __ldcs((const uint4 *)pp.g[q] + vec);
            const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
            for (int e = 0; e < 8; e++) {
                const float x = h2f_bits_dp((e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu));
                s[e] = q == 0 ? x : __fadd_rn(s[e], x);
            }
        }
    }
    float4 w0 = __ldcs(w32 + 2 * j), w1 = __ldcs(w32 + 2 * j + 1);
    float4 v0 = make_float4(0, 0, 0, 0), v1 = v0;
    if (MOM) { v0 = __ldcs(v + 2 * j); v1 = __ldcs(v + 2 * j + 1); }
    bool bad = false;
    float *wf[2] = {&w0.x, &w1.x}, *vf[2] = {&v0.x, &v1.x};
#pragma unroll
    for (int e = 0; e < 8; e++) dp_elem<MOM>(s[e], inv, lr, mu, wf[e >> 2][e & 3], vf[e >> 2][e & 3], bad);
    uint4 h;
    h.x = f2h_bits_dp(w0.x) | (f2h_bits_dp(w0.y) << 16);
    h.y = f2h_bits_dp(w0.z) | (f2h_bits_dp(w0.w) << 16);
    h.z = f2h_bits_dp(w1.x) | (f2h_bits_dp(w1.y) << 16);
    h.w = f2h_bits_dp(w1.z) | (f2h_bits_dp(w1.w) << 16);
    __stcs(w32 + 2 * j, w0);
    __stcs(w32 + 2 * j + 1, w1);
    if (MOM) { __stcs(v + 2 * j, v0); __stcs(v + 2 * j + 1, v1); }
    if (RT) {
#pragma unroll
        for (int q = 0; q < RT; q++) __stcs((uint4 *)pp.w[q] + vec, h);
    } else {
        for (int q = 0; q < R; q++) __stcs((uint4 *)pp.w[q] + vec, h);
    }
    if (__any_sync(__activemask(), bad) && (threadIdx.x & 31) == 0) atomicOr(flags + 1, 1u);
}

// the up to seven elements after the last whole vector of a shard (one warp)
template <bool MOM>
__global__ void k_dp_step_tail(const DpPeers pp, int R, float *__restrict__ w32, float *__restrict__ v, size_t first,
                               size_t begin, size_t count, float inv, const float *__restrict__ S_dev, float lr, float mu,
                               uint32_t *flags)
{
    pdl_trigger();
    pdl_wait();
    if (S_dev) inv = __fdiv_rn(1.0f, __fmul_rn(*S_dev, (float)R));
    if (any_replica_overflowed(pp, R)) {
        if (threadIdx.x == 0) atomicOr(flags, 1u);
        return;
    }
    bool bad = false;
    for (size_t i = begin + threadIdx.x; i < count; i += blockDim.x) {
        float s = h2f_bits_dp(pp.g[0][first + i]);
        for (int q = 1; q < R; q++) s = __fadd_rn(s, h2f_bits_dp(pp.g[q][first + i]));
        float w = w32[i], m = MOM ? v[i] : 0.0f;
        dp_elem<MOM>(s, inv, lr, mu, w, m, bad);
        w32[i] = w;
        if (MOM) v[i] = m;
        const uint16_t h = (uint16_t)f2h_bits_dp(w);
        for (int q = 0; q < R; q++) pp.w[q][first + i] = h;
    }
    if (bad) atomicOr(flags + 1, 1u);
}

// The same exchange with the other optimizer steps (weight decay, Nesterov, Adagrad, Adam) on the
// mean gradient: replica count at run time, states s1 / s2 of the shard (s2: Adam only).
template <int KIND, bool WD>
__global__ void __launch_bounds__(kDpThreads) k_dp_step_opt(const DpPeers pp, int R, float4 *__restrict__ w32,
                                                            float4 *__restrict__ s1p, float4 *__restrict__ s2p, size_t first,
                                                            size_t n8, float inv, const float *__restrict__ S_dev, float lr,
                                                            float mu, float b2, float eps, float wd, float b1t, float b2t,
                                                            const float *__restrict__ betat_dev, uint32_t *flags,
                                                            const float *__restrict__ coef_dev,
                                                            const float4 *__restrict__ sum32)
{
    pdl_trigger();
    pdl_wait();
    if (S_dev) inv = __fdiv_rn(1.0f, __fmul_rn(*S_dev, (float)R));
    if (any_replica_overflowed(pp, R)) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(flags, 1u);
        return;
    }
    const float coef = coef_dev ? *coef_dev : 1.0f;      // global-norm clipping of the mean gradient (1 = off)
    const size_t j = (size_t)blockIdx.x * kDpThreads + threadIdx.x;
    if (j >= n8) return;
    if (betat_dev) { b1t = __fmul_rn(betat_dev[0], mu); b2t = __fmul_rn(betat_dev[1], b2); }
    const float bc1 = __fsub_rn(1.0f, b1t), bc2 = __fsub_rn(1.0f, b2t);
    const float omb1 = __fsub_rn(1.0f, mu), omb2 = __fsub_rn(1.0f, b2);
    const bool use_s1 = KIND != MPT_OPT_SGD || mu != 0.0f;
    constexpr bool S2 = KIND == MPT_OPT_ADAM;
    const size_t vec = first / 8 + j;
    float s[8];
    if (sum32) {      // the FP32 sums over the replicas were formed earlier (k_dp_reduce), in the same order
        const float4 x0 = __ldcs(sum32 + 2 * j), x1 = __ldcs(sum32 + 2 * j + 1);
        s[0] = x0.x; s[1] = x0.y; s[2] = x0.z; s[3] = x0.w; s[4] = x1.x; s[5] = x1.y; s[6] = x1.z; s[7] = x1.w;
    } else {
#pragma unroll 4
        for (int q = 0; q < R; q++) {
            const uint4 g = __ldcs((const uint4 *)pp.g[q] + vec);
            const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
            for (int e = 0; e < 8; e++) {
                const float x = h2f_bits_dp((e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu));
                s[e] = q == 0 ? x : __fadd_rn(s[e], x);
            }
        }
    }
    float4 w0 = __ldcs(w32 + 2 * j), w1 = __ldcs(w32 + 2 * j + 1);
    float4 a0 = make_float4(0, 0, 0, 0), a1 = a0, b0 = a0, b1 = a0;
    if (use_s1) { a0 = __ldcs(s1p + 2 * j); a1 = __ldcs(s1p + 2 * j + 1); }
    if (S2) { b0 = __ldcs(s2p + 2 * j); b1 = __ldcs(s2p + 2 * j + 1); }
    bool bad = false;
    float *wf[2] = {&w0.x, &w1.x}, *af[2] = {&a0.x, &a1.x}, *bf[2] = {&b0.x, &b1.x};
#pragma unroll
    for (int e = 0; e < 8; e++)
        opt1<KIND, WD>(s[e], wf[e >> 2][e & 3], af[e >> 2][e & 3], bf[e >> 2][e & 3], inv, lr, mu, b2, omb1, omb2, eps, wd,
                       bc1, bc2, coef, bad);
    uint4 h;
    h.x = f2h_bits_dp(w0.x) | (f2h_bits_dp(w0.y) << 16);
    h.y = f2h_bits_dp(w0.z) | (f2h_bits_dp(w0.w) << 16);
    h.z = f2h_bits_dp(w1.x) | (f2h_bits_dp(w1.y) << 16);
    h.w = f2h_bits_dp(w1.z) | (f2h_bits_dp(w1.w) << 16);
    __stcs(w32 + 2 * j, w0);
    __stcs(w32 + 2 * j + 1, w1);
    if (use_s1) { __stcs(s1p + 2 * j, a0); __stcs(s1p + 2 * j + 1, a1); }
    if (S2) { __stcs(s2p + 2 * j, b0); __stcs(s2p + 2 * j + 1, b1); }
    for (int q = 0; q < R; q++) __stcs((uint4 *)pp.w[q] + vec, h);
    if (__any_sync(__activemask(), bad) && (threadIdx.x & 31) == 0) atomicOr(flags + 1, 1u);
}

template <int KIND, bool WD>
__global__ void k_dp_step_opt_tail(const DpPeers pp, int R, float *__restrict__ w32, float *__restrict__ s1p,
                                   float *__restrict__ s2p, size_t first, size_t begin, size_t count, float inv,
                                   const float *__restrict__ S_dev, float lr, float mu, float b2, float eps, float wd,
                                   float b1t, float b2t, const float *__restrict__ betat_dev, uint32_t *flags,
                                   const float *__restrict__ coef_dev, const float *__restrict__ sum32)
{
    pdl_trigger();
    pdl_wait();
    if (S_dev) inv = __fdiv_rn(1.0f, __fmul_rn(*S_dev, (float)R));
    if (any_replica_overflowed(pp, R)) {
        if (threadIdx.x == 0) atomicOr(flags, 1u);
        return;
    }
    const float coef = coef_dev ? *coef_dev : 1.0f;
    if (betat_dev) { b1t = __fmul_rn(betat_dev[0], mu); b2t = __fmul_rn(betat_dev[1], b2); }
    const float bc1 = __fsub_rn(1.0f, b1t), bc2 = __fsub_rn(1.0f, b2t);
    const float omb1 = __fsub_rn(1.0f, mu), omb2 = __fsub_rn(1.0f, b2);
    const bool use_s1 = KIND != MPT_OPT_SGD || mu != 0.0f;
    bool bad = false;
    for (size_t i = begin + threadIdx.x; i < count; i += blockDim.x) {
        float s;
        if (sum32) {
            s = sum32[i];
        } else {
            s = h2f_bits_dp(pp.g[0][first + i]);
            for (int q = 1; q < R; q++) s = __fadd_rn(s, h2f_bits_dp(pp.g[q][first + i]));
        }
        float w = w32[i], a = use_s1 ? s1p[i] : 0.0f, b = KIND == MPT_OPT_ADAM ? s2p[i] : 0.0f;
        opt1<KIND, WD>(s, w, a, b, inv, lr, mu, b2, omb1, omb2, eps, wd, bc1, bc2, coef, bad);
        w32[i] = w;
        if (use_s1) s1p[i] = a;
        if (KIND == MPT_OPT_ADAM) s2p[i] = b;
        const uint16_t h = (uint16_t)f2h_bits_dp(w);
        for (int q = 0; q < R; q++) pp.w[q][first + i] = h;
    }
    if (bad) atomicOr(flags + 1, 1u);
}

template <int KIND, bool WD>
cudaError_t launch_dp_opt(const DpPeers &pp, int R, float *w32, float *s1, float *s2, size_t first, size_t count, float inv,
                          const float *S_dev, float lr, float mu, float b2, float eps, float wd, float b1t, float b2t,
                          const float *betat_dev, uint32_t *flags, cudaStream_t st, int *n_launches, const float *coef_dev,
                          const float *sum32)
{
    const size_t n8 = count / 8;
    if (n_launches) *n_launches = (n8 ? 1 : 0) + (n8 * 8 < count || count == 0 ? 1 : 0);
    if (n8)
        MPT_LAUNCH(k_dp_step_opt<KIND, WD>, dim3((unsigned)((n8 + kDpThreads - 1) / kDpThreads)), dim3(kDpThreads), 0, st, pp, R,
                   (float4 *)w32, (float4 *)s1, (float4 *)s2, first, n8, inv, S_dev, lr, mu, b2, eps, wd, b1t, b2t, betat_dev,
                   flags, coef_dev, (const float4 *)sum32);
    if (n8 * 8 < count || count == 0)
        MPT_LAUNCH(k_dp_step_opt_tail<KIND, WD>, dim3(1), dim3(32), 0, st, pp, R, w32, s1, s2, first, n8 * 8, count, inv, S_dev,
                   lr, mu, b2, eps, wd, b1t, b2t, betat_dev, flags, coef_dev, sum32);
    return cudaGetLastError();
}

// First half of the exchange by itself: the FP32 sum over the replicas, in replica order, of the elements
// [first, first + count) of their FP16 gradient arrays (first and count multiples of 8), stored raw.  The
// step kernels take such sums in place of the gradients (their sum32 argument), so the pull over the link
// can run per layer beside the rest of the backward pass and the update after the overflow is known.
__global__ void __launch_bounds__(kDpThreads) k_dp_reduce(const DpPeers pp, int R, size_t first, size_t n8, float4 *__restrict__ out)
{
    pdl_trigger();
    pdl_wait();
    const size_t j = (size_t)blockIdx.x * kDpThreads + threadIdx.x;
    if (j >= n8) return;
    const size_t vec = first / 8 + j;
    float s[8];
#pragma unroll 4
    for (int q = 0; q < R; q++) {
        const uint4 g = __ldcs((const uint4 *)pp.g[q] + vec);
        const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
        for (int e = 0; e < 8; e++) {
            const float x = h2f_bits_dp((e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu));
            s[e] = q == 0 ? x : __fadd_rn(s[e], x);
        }
    }
    out[2 * j] = make_float4(s[0], s[1], s[2], s[3]);
    out[2 * j + 1] = make_float4(s[4], s[5], s[6], s[7]);
}

// ---- global-norm clipping of the mean gradient (section 3.2): sum of squares of this replica's shard
// of the mean unscaled gradient in double over a fixed partition (same tree as the single-GPU norm),
// combined into one double that the replica publishes; then every replica adds all replicas' doubles
// in ascending replica order and forms the same coefficient.
constexpr int kDpNormParts = 592;

__device__ __forceinline__ double dp_block_sum_fixed(double v, double *sh)
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

__global__ void __launch_bounds__(kDpThreads) k_dp_sqnorm(const DpPeers pp, int R, size_t first, size_t count, float inv,
                                                          const float *__restrict__ S_dev, double *__restrict__ parts,
                                                          const float *__restrict__ sum32)
{
    pdl_trigger();
    pdl_wait();
    __shared__ double sh[kDpThreads / 32];
    if (S_dev) inv = __fdiv_rn(1.0f, __fmul_rn(*S_dev, (float)R));
    double acc = 0.0;
    const size_t n8 = count / 8, stride = (size_t)gridDim.x * kDpThreads;
    for (size_t j = (size_t)blockIdx.x * kDpThreads + threadIdx.x; j < n8; j += stride) {
        const size_t vec = first / 8 + j;
        float s[8];
        if (sum32) {      // sums formed earlier by k_dp_reduce
            const float4 x0 = __ldcs((const float4 *)sum32 + 2 * j), x1 = __ldcs((const float4 *)sum32 + 2 * j + 1);
            s[0] = x0.x; s[1] = x0.y; s[2] = x0.z; s[3] = x0.w; s[4] = x1.x; s[5] = x1.y; s[6] = x1.z; s[7] = x1.w;
        } else {
            for (int q = 0; q < R; q++) {
                const uint4 g = __ldcs((const uint4 *)pp.g[q] + vec);
                const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
                for (int e = 0; e < 8; e++) {
                    const float x = h2f_bits_dp((e & 1) ? (gw[e >> 1] >> 16) : (gw[e >> 1] & 0xFFFFu));
                    s[e] = q == 0 ? x : __fadd_rn(s[e], x);
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 8; e++) {
            const double v = (double)__fmul_rn(s[e], inv);
            acc += v * v;
        }
    }
    if (blockIdx.x == 0)      // the up to seven elements after the shard's last whole vector
        for (size_t i = n8 * 8 + threadIdx.x; i < count; i += kDpThreads) {
            float s;
            if (sum32) {
                s = sum32[i];
            } else {
                s = h2f_bits_dp(pp.g[0][first + i]);
                for (int q = 1; q < R; q++) s = __fadd_rn(s, h2f_bits_dp(pp.g[q][first + i]));
            }
            const double v = (double)__fmul_rn(s, inv);
            acc += v * v;
        }
    const double total = dp_block_sum_fixed(acc, sh);
    if (threadIdx.x == 0) parts[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) k_dp_norm_publish(const double *__restrict__ parts, int nparts, double *slot)
{
    pdl_trigger();
    pdl_wait();
    __shared__ double sh[32];
    double acc = 0.0;
    for (int i = threadIdx.x; i < nparts; i += 1024) acc += parts[i];
    const double total = dp_block_sum_fixed(acc, sh);
    if (threadIdx.x == 0) *slot = total;
}

struct DpNormPeers {
    const double *slot[MPT_DP_MAX_REPLICAS];
};

// out[0] = coef = min(1, clip / (sqrt(total) + 1e-6)) rounded to FP32, out[1] = norm (FP32);
// total = the replicas' shard sums added in ascending replica order.
__global__ void k_dp_clip_coef(const DpNormPeers np, int R, float clip, float *out)
{
    pdl_trigger();
    pdl_wait();
    double total = 0.0;
    for (int q = 0; q < R; q++) total += *(volatile const double *)np.slot[q];
    const double norm = sqrt(total);
    out[0] = (float)fmin(1.0, (double)clip / (norm + 1e-6));
    out[1] = (float)norm;
}

template <bool MOM>
cudaError_t launch_dp(const DpPeers &pp, int R, float *w32, float *v, size_t first, size_t count, float inv,
                      const float *S_dev, float lr, float mu, uint32_t *flags, cudaStream_t st, int *n_launches)
{
    if (n_launches) *n_launches = (count / 8 ? 1 : 0) + ((count / 8) * 8 < count || count == 0 ? 1 : 0);
    const size_t n8 = count / 8;
    if (n8) {
        const dim3 grid((unsigned)((n8 + kDpThreads - 1) / kDpThreads)), block(kDpThreads);
        switch (R) {
            case 2: MPT_LAUNCH(k_dp_step<2, MOM>, grid, block, 0, st, pp, R, (float4 *)w32, (float4 *)v, first, n8, inv, S_dev, lr, mu, flags); break;
            case 4: MPT_LAUNCH(k_dp_step<4, MOM>, grid, block, 0, st, pp, R, (float4 *)w32, (float4 *)v, first, n8, inv, S_dev, lr, mu, flags); break;
            case 8: MPT_LAUNCH(k_dp_step<8, MOM>, grid, block, 0, st, pp, R, (float4 *)w32, (float4 *)v, first, n8, inv, S_dev, lr, mu, flags); break;
            default: MPT_LAUNCH(k_dp_step<0, MOM>, grid, block, 0, st, pp, R, (float4 *)w32, (float4 *)v, first, n8, inv, S_dev, lr, mu, flags); break;
        }
    }
    // also for an empty shard: the launch then only publishes the skip decision in this replica's flags
    if (n8 * 8 < count || count == 0)
        MPT_LAUNCH(k_dp_step_tail<MOM>, dim3(1), dim3(32), 0, st, pp, R, w32, v, first, n8 * 8, count, inv, S_dev, lr, mu, flags);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_dp_step(const uint16_t *const *g16, const uint32_t *const *flag, uint16_t *const *w16, int R,
                           float *w32_shard, float *v_shard, size_t first, size_t count, float inv_SR, const float *S_dev,
                           float lr, float mu, uint32_t *flags, cudaStream_t st, int *n_launches)
{
    DpPeers pp = {};
    for (int q = 0; q < R; q++) {
        pp.g[q] = g16[q];
        pp.flag[q] = flag[q];
        pp.w[q] = w16[q];
    }
    return mu != 0.0f ? launch_dp<true>(pp, R, w32_shard, v_shard, first, count, inv_SR, S_dev, lr, mu, flags, st, n_launches)
                      : launch_dp<false>(pp, R, w32_shard, nullptr, first, count, inv_SR, S_dev, lr, mu, flags, st, n_launches);
}

cudaError_t launch_dp_step_opt(int kind, const uint16_t *const *g16, const uint32_t *const *flag, uint16_t *const *w16, int R,
                               float *w32_shard, float *s1_shard, float *s2_shard, size_t first, size_t count, float inv_SR,
                               const float *S_dev, float lr, float mu, float b2, float eps, float wd, float b1t, float b2t,
                               const float *betat_dev, uint32_t *flags, cudaStream_t st, int *n_launches,
                               const float *coef_dev, const float *sum32)
{
    DpPeers pp = {};
    for (int q = 0; q < R; q++) {
        pp.g[q] = g16[q];
        pp.flag[q] = flag[q];
        pp.w[q] = w16[q];
    }
#define MPT_DP_OPT(KIND)                                                                                                    \
    (wd != 0.0f ? launch_dp_opt<KIND, true>(pp, R, w32_shard, s1_shard, s2_shard, first, count, inv_SR, S_dev, lr, mu, b2, eps, \
                                            wd, b1t, b2t, betat_dev, flags, st, n_launches, coef_dev, sum32)                 \
                : launch_dp_opt<KIND, false>(pp, R, w32_shard, s1_shard, s2_shard, first, count, inv_SR, S_dev, lr, mu, b2,   \
                                             eps, wd, b1t, b2t, betat_dev, flags, st, n_launches, coef_dev, sum32))
    switch (kind) {
        case MPT_OPT_SGD: return MPT_DP_OPT(MPT_OPT_SGD);
        case MPT_OPT_NESTEROV: return MPT_DP_OPT(MPT_OPT_NESTEROV);
        case MPT_OPT_ADAGRAD: return MPT_DP_OPT(MPT_OPT_ADAGRAD);
        case MPT_OPT_ADAM: return MPT_DP_OPT(MPT_OPT_ADAM);
        default: return cudaErrorInvalidValue;
    }
#undef MPT_DP_OPT
}

cudaError_t launch_dp_reduce(const uint16_t *const *g16, int R, size_t first, size_t count, float *sum32_out, cudaStream_t st)
{
    if ((first | count) & 7) return cudaErrorInvalidValue;
    if (count == 0) return cudaSuccess;
    DpPeers pp = {};
    for (int q = 0; q < R; q++) pp.g[q] = g16[q];
    const size_t n8 = count / 8;
    MPT_LAUNCH(k_dp_reduce, dim3((unsigned)((n8 + kDpThreads - 1) / kDpThreads)), dim3(kDpThreads), 0, st, pp, R, first, n8,
               (float4 *)sum32_out);
    return cudaGetLastError();
}

cudaError_t launch_dp_sqnorm(const uint16_t *const *g16, int R, size_t first, size_t count, float inv_SR, const float *S_dev,
                             double *parts, double *slot, cudaStream_t st, const float *sum32)
{
    DpPeers pp = {};
    for (int q = 0; q < R; q++) pp.g[q] = g16[q];
    size_t want = (count / 8 + kDpThreads - 1) / kDpThreads;
    const int grid = (int)(want < 1 ? 1 : (want > (size_t)kDpNormParts ? (size_t)kDpNormParts : want));
    MPT_LAUNCH(k_dp_sqnorm, dim3(grid), dim3(kDpThreads), 0, st, pp, R, first, count, inv_SR, S_dev, parts, sum32);
    MPT_LAUNCH(k_dp_norm_publish, dim3(1), dim3(1024), 0, st, (const double *)parts, grid, slot);
    return cudaGetLastError();
}

cudaError_t launch_dp_clip_coef(const double *const *slots, int R, float clip, float *out2, cudaStream_t st)
{
    DpNormPeers np = {};
    for (int q = 0; q < R; q++) np.slot[q] = slots[q];
    MPT_LAUNCH(k_dp_clip_coef, dim3(1), dim3(1), 0, st, np, R, clip, out2);
    return cudaGetLastError();
}

}  // namespace mpt

using namespace mpt;

extern "C" {

int mpt_dp_shard(size_t n, int R, int rank, size_t *lo_out, size_t *hi_out)
{
    if (R < 1 || R > MPT_DP_MAX_REPLICAS || rank < 0 || rank >= R || !lo_out || !hi_out) return MPT_ERR_INVALID_ARG;
    const size_t vecs = (n + 7) / 8;
    const size_t per = ((vecs + (size_t)R - 1) / (size_t)R) * 8;
    size_t lo = per * (size_t)rank, hi = lo + per;
    if (lo > n) lo = n;
    if (hi > n) hi = n;
    *lo_out = lo;
    *hi_out = hi;
    return MPT_OK;
}

int mpt_dp_step_flat(const uint16_t *const *g16_peers, const uint32_t *const *flag_peers, uint16_t *const *w16_peers,
                     float *w32_shard_dev, float *v_shard_dev, size_t n, int R, int rank, float S, float lr, float mu,
                     uint32_t *flags_dev, void *cuda_stream)
{
    if (!g16_peers || !flag_peers || !w16_peers || !flags_dev) return MPT_ERR_INVALID_ARG;
    size_t lo = 0, hi = 0;
    if (mpt_dp_shard(n, R, rank, &lo, &hi) != MPT_OK) return MPT_ERR_INVALID_ARG;
    if (!(S > 0.0f) || !(lr == lr) || !(mu == mu)) return MPT_ERR_INVALID_ARG;
    const bool mom = mu != 0.0f;
    for (int q = 0; q < R; q++) {
        if (!g16_peers[q] || !flag_peers[q] || !w16_peers[q]) return MPT_ERR_INVALID_ARG;
        if ((((uintptr_t)g16_peers[q] | (uintptr_t)w16_peers[q]) & 15) != 0 || ((uintptr_t)flag_peers[q] & 3) != 0)
            return MPT_ERR_INVALID_ARG;
    }
    const size_t count = hi - lo;
    if (count && (!w32_shard_dev || (mom && !v_shard_dev))) return MPT_ERR_INVALID_ARG;
    if (count && (((uintptr_t)w32_shard_dev | (uintptr_t)v_shard_dev) & 15) != 0) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemsetAsync(flags_dev + 1, 0, sizeof(uint32_t), st);
    if (e != cudaSuccess) return MPT_ERR_CUDA;
    const float inv = 1.0f / (S * (float)R);
    e = launch_dp_step(g16_peers, flag_peers, w16_peers, R, w32_shard_dev, v_shard_dev, lo, count, inv, nullptr, lr, mu, flags_dev,
                       st, nullptr);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_dp_norm_flat(const uint16_t *const *g16_peers, size_t n, int R, int rank, float S, void *scratch_dev,
                     double *norm_slot_dev, void *cuda_stream)
{
    if (!g16_peers || !scratch_dev || !norm_slot_dev) return MPT_ERR_INVALID_ARG;
    size_t lo = 0, hi = 0;
    if (mpt_dp_shard(n, R, rank, &lo, &hi) != MPT_OK) return MPT_ERR_INVALID_ARG;
    if (!(S > 0.0f)) return MPT_ERR_INVALID_ARG;
    for (int q = 0; q < R; q++)
        if (!g16_peers[q] || ((uintptr_t)g16_peers[q] & 15) != 0) return MPT_ERR_INVALID_ARG;
    if ((((uintptr_t)scratch_dev | (uintptr_t)norm_slot_dev) & 7) != 0) return MPT_ERR_INVALID_ARG;
    const float inv = 1.0f / (S * (float)R);
    return launch_dp_sqnorm(g16_peers, R, lo, hi - lo, inv, nullptr, (double *)scratch_dev, norm_slot_dev,
                            (cudaStream_t)cuda_stream) == cudaSuccess
               ? MPT_OK
               : MPT_ERR_CUDA;
}

int mpt_dp_step_flat_opt(const mpt_optimizer *opt, const uint16_t *const *g16_peers, const uint32_t *const *flag_peers,
                         uint16_t *const *w16_peers, float *w32_shard_dev, float *s1_shard_dev, float *s2_shard_dev, size_t n,
                         int R, int rank, float S, float b1t, float b2t, uint32_t *flags_dev, const double *const *norm_peers,
                         float *clip_out_dev, void *cuda_stream)
{
    if (!opt || !g16_peers || !flag_peers || !w16_peers || !flags_dev) return MPT_ERR_INVALID_ARG;
    if (opt->kind < MPT_OPT_SGD || opt->kind > MPT_OPT_ADAM || !(opt->clip_norm >= 0.0f)) return MPT_ERR_INVALID_ARG;
    const bool clip = opt->clip_norm > 0.0f;
    if (clip) {
        if (!norm_peers || !clip_out_dev || R < 1 || R > MPT_DP_MAX_REPLICAS) return MPT_ERR_INVALID_ARG;
        for (int q = 0; q < R; q++)
            if (!norm_peers[q] || ((uintptr_t)norm_peers[q] & 7) != 0) return MPT_ERR_INVALID_ARG;
    }
    size_t lo = 0, hi = 0;
    if (mpt_dp_shard(n, R, rank, &lo, &hi) != MPT_OK) return MPT_ERR_INVALID_ARG;
    if (!(S > 0.0f) || !(opt->lr == opt->lr)) return MPT_ERR_INVALID_ARG;
    for (int q = 0; q < R; q++) {
        if (!g16_peers[q] || !flag_peers[q] || !w16_peers[q]) return MPT_ERR_INVALID_ARG;
        if ((((uintptr_t)g16_peers[q] | (uintptr_t)w16_peers[q]) & 15) != 0 || ((uintptr_t)flag_peers[q] & 3) != 0)
            return MPT_ERR_INVALID_ARG;
    }
    const size_t count = hi - lo;
    const bool need1 = opt->kind != MPT_OPT_SGD || opt->momentum != 0.0f, need2 = opt->kind == MPT_OPT_ADAM;
    if (count && (!w32_shard_dev || (need1 && !s1_shard_dev) || (need2 && !s2_shard_dev))) return MPT_ERR_INVALID_ARG;
    if (count && (((uintptr_t)w32_shard_dev | (uintptr_t)s1_shard_dev | (uintptr_t)s2_shard_dev) & 15) != 0) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemsetAsync(flags_dev + 1, 0, sizeof(uint32_t), st);
    if (e != cudaSuccess) return MPT_ERR_CUDA;
    const float inv = 1.0f / (S * (float)R);
    if (clip && launch_dp_clip_coef(norm_peers, R, opt->clip_norm, clip_out_dev, st) != cudaSuccess) return MPT_ERR_CUDA;
    e = launch_dp_step_opt(opt->kind, g16_peers, flag_peers, w16_peers, R, w32_shard_dev, s1_shard_dev, s2_shard_dev, lo, count, inv,
                           nullptr, opt->lr, opt->momentum, opt->beta2, opt->eps, opt->weight_decay, b1t, b2t, nullptr, flags_dev, st,
                           nullptr, clip ? clip_out_dev : nullptr);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_dp_alloc(size_t bytes, void **dev_ptr_out)
{
    if (!dev_ptr_out || bytes == 0) return MPT_ERR_INVALID_ARG;
    *dev_ptr_out = nullptr;
    return cudaMalloc(dev_ptr_out, bytes) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_dp_free(void *dev_ptr)
{
    if (!dev_ptr) return MPT_ERR_INVALID_ARG;
    return cudaFree(dev_ptr) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_dp_export(const void *dev_ptr, uint8_t *handle_out)
{
    static_assert(sizeof(cudaIpcMemHandle_t) == MPT_DP_HANDLE_BYTES, "handle size");
    if (!dev_ptr || !handle_out) return MPT_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    if (cudaIpcGetMemHandle(&h, const_cast<void *>(dev_ptr)) != cudaSuccess) return MPT_ERR_CUDA;
    memcpy(handle_out, &h, sizeof(h));
    return MPT_OK;
}

int mpt_dp_open(const uint8_t *handle, void **dev_ptr_out)
{
    if (!handle || !dev_ptr_out) return MPT_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle, sizeof(h));
    *dev_ptr_out = nullptr;
    return cudaIpcOpenMemHandle(dev_ptr_out, h, cudaIpcMemLazyEnablePeerAccess) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_dp_close(void *dev_ptr)
{
    if (!dev_ptr) return MPT_ERR_INVALID_ARG;
    return cudaIpcCloseMemHandle(dev_ptr) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

}  // extern "C"

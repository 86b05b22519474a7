// Fused softmax cross-entropy forward + loss-scaled backward (paper sections 3.2, 3.3):
// FP16 logits in, FP32 max / sum-of-exponentials / log, FP16 logit gradient out with
// the factor S/B applied.  One CTA per row; the row is read from HBM once and written
// once: 4 bytes per logit.  Rows of up to 65536 classes with 16-byte aligned pitches stay
// in registers (k_softmax_ce_reg); other rows go through shared memory or are re-read
// (k_softmax_ce).
#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

static constexpr int kMaxSmemRowBytes = 200 * 1024;

__device__ __forceinline__ float hbits2f(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }
__device__ __forceinline__ uint32_t f2hbits(float x) { return (uint32_t)__half_as_ushort(__float2half_rn(x)); }

// 2^x on the special-function unit, one instruction: results below 2^-126 flush to zero (such a
// term is 10^-38 of a sum that is at least 1), NaN and the infinities behave as in exp2f.
__device__ __forceinline__ float ex2_ftz(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float block_reduce(float v, bool is_max, float *red)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float other = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = is_max ? fmaxf(v, other) : v + other;
    }
    __syncthreads();  // protect red[] from the previous use
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < nw; w++) r = is_max ? fmaxf(r, red[w]) : r + red[w];   // fixed order
    return r;
}

// VEC: rows are 16-byte aligned and C % 8 == 0 is NOT required (tail handled scalar).
// CACHE: the row fits the dynamic shared-memory buffer.
template <bool VEC, bool CACHE>
__global__ void __launch_bounds__(1024) k_softmax_ce(const uint16_t *__restrict__ z, int ldz,
                                                     const int32_t *__restrict__ labels, int B, int C, float c,
                                                     uint16_t *dz, int lddz, float *__restrict__ row_loss,
                                                     uint32_t *bad_labels, const float *__restrict__ scale_dev)
{
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(16) uint16_t srow[];
    if (scale_dev) c = __fdiv_rn(*scale_dev, (float)B);
    __shared__ float red[32];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int C8 = VEC ? (C / 8) : 0;

    for (int row = blockIdx.x; row < B; row += gridDim.x) {
        const uint16_t *zr = z + (size_t)row * ldz;
        uint16_t *dr = dz + (size_t)row * lddz;
        const int y = labels[row];
        if (y < 0 || y >= C) {  // contributes neither loss nor gradient
            for (int j = tid; j < C; j += nt) dr[j] = 0;
            if (tid == 0) {
                row_loss[row] = 0.0f;
                if (bad_labels) atomicAdd(bad_labels, 1u);
            }
            continue;
        }
        // pass 1: read the row once, keep it on chip, running max
        float m = -INFINITY;
        if (VEC) {
            const uint4 *zv = (const uint4 *)zr;
            for (int i = tid; i < C8; i += nt) {
                uint4 x = __ldcs(zv + i);
                if (CACHE) ((uint4 *)srow)[i] = x;
                uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    m = fmaxf(m, hbits2f(w[q] & 0xFFFFu));
                    m = fmaxf(m, hbits2f(w[q] >> 16));
                }
            }
        }
        for (int j = C8 * 8 + tid; j < C; j += nt) {
            uint16_t h = zr[j];
            if (CACHE) srow[j] = h;
            m = fmaxf(m, hbits2f(h));
        }
        m = block_reduce(m, true, red);   // also orders the srow writes before the reads below

        // pass 2: sum of exponentials in FP32
        float s = 0.0f;
        for (int j = tid; j < C; j += nt) {
            float v = hbits2f(CACHE ? srow[j] : zr[j]);
            s += expf(v - m);
        }
        s = block_reduce(s, false, red);
        if (tid == 0) {
            float zy = hbits2f(CACHE ? srow[y] : zr[y]);
            row_loss[row] = (m + logf(s)) - zy;
        }
        // pass 3: gradient (e/s - onehot) * c, rounded to FP16
        if (VEC) {
            uint4 *dv = (uint4 *)dr;
            for (int i = tid; i < C8; i += nt) {
                uint4 x = CACHE ? ((const uint4 *)srow)[i] : ((const uint4 *)zr)[i];
                uint32_t w[4] = {x.x, x.y, x.z, x.w};
                uint32_t o[4];
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    int j = i * 8 + q * 2;
                    float p0 = __fdiv_rn(expf(hbits2f(w[q] & 0xFFFFu) - m), s);
                    float p1 = __fdiv_rn(expf(hbits2f(w[q] >> 16) - m), s);
                    float d0 = __fmul_rn(__fsub_rn(p0, (j == y) ? 1.0f : 0.0f), c);
                    float d1 = __fmul_rn(__fsub_rn(p1, (j + 1 == y) ? 1.0f : 0.0f), c);
                    o[q] = f2hbits(d0) | (f2hbits(d1) << 16);
                }
                __stcs(dv + i, make_uint4(o[0], o[1], o[2], o[3]));
            }
        }
        for (int j = C8 * 8 + tid; j < C; j += nt) {
            float p = __fdiv_rn(expf(hbits2f(CACHE ? srow[j] : zr[j]) - m), s);
            dr[j] = (uint16_t)f2hbits(__fmul_rn(__fsub_rn(p, (j == y) ? 1.0f : 0.0f), c));
        }
        __syncthreads();  // srow is reused by the next row
    }
}

// Register-resident variant: thread t holds the 8-element vectors t, t + T, t + 2T, ... of its
// row (T = blockDim.x, at most VPT of them) and, for rows whose length is not a multiple of 8,
// threads 0..6 hold one tail element each.  Exponentials are 2^((z - m) * log2 e) on the
// special-function unit: z - m is exact near the maximum, so the rounding of the argument
// only touches terms far below it, and is far below FP16 resolution after the store.  Non-label outputs are e_j * (c / s); the label's output is
// (e_y / s - 1) * c, evaluated separately because of the cancellation.
template <int VPT>
__global__ void __launch_bounds__(1024, VPT <= 4 ? 2 : 1) k_softmax_ce_reg(const uint16_t *__restrict__ z, int ldz,
                                                         const int32_t *__restrict__ labels, int C, float c,
                                                         uint16_t *__restrict__ dz, int lddz,
                                                         float *__restrict__ row_loss, uint32_t *bad_labels,
                                                         const float *__restrict__ scale_dev)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    if (scale_dev) c = __fdiv_rn(*scale_dev, (float)gridDim.x);   // one CTA per row: gridDim.x is the batch
    const int tid = threadIdx.x, nt = blockDim.x, row = blockIdx.x;
    const int C8 = C >> 3, tail = C & 7;
    const uint16_t *zr = z + (size_t)row * ldz;
    uint16_t *dr = dz + (size_t)row * lddz;
    const int y = labels[row];
    if (y < 0 || y >= C) {  // contributes neither loss nor gradient
        for (int j = tid; j < C; j += nt) dr[j] = 0;
        if (tid == 0) {
            row_loss[row] = 0.0f;
            if (bad_labels) atomicAdd(bad_labels, 1u);
        }
        return;
    }
    constexpr float LOG2E = 1.4426950408889634f;
    uint4 x[VPT];
#pragma unroll
    for (int u = 0; u < VPT; u++) {
        const int i = tid + u * nt;
        if (i < C8) x[u] = __ldcs((const uint4 *)zr + i);
    }
    float tv = 0.0f;
    const bool has_tail = tid < tail;
    if (has_tail) tv = hbits2f(zr[C8 * 8 + tid]);

    float m = -INFINITY;
#pragma unroll
    for (int u = 0; u < VPT; u++) {
        if (tid + u * nt < C8) {
            const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
            for (int q = 0; q < 4; q++) m = fmaxf(m, fmaxf(hbits2f(w[q] & 0xFFFFu), hbits2f(w[q] >> 16)));
        }
    }
    if (has_tail) m = fmaxf(m, tv);
    m = block_reduce(m, true, red);

    // one FMA and one special-function instruction per logit: 2^(z*log2e - mL), mL = rn(m*log2e);
    // the factor 2^delta this puts on every exponential of the row (delta = m*log2e - mL, exact by
    // an FMA) cancels in e/s and is taken out of log(s)
    const float mL = __fmul_rn(m, LOG2E);
    const float delta = fmaf(m, LOG2E, -mL);
    float s = 0.0f;
#pragma unroll
    for (int u = 0; u < VPT; u++) {
        if (tid + u * nt < C8) {
            const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
            for (int q = 0; q < 4; q++) {
                const float2 f = __half22float2(*(const __half2 *)&w[q]);
                s += ex2_ftz(fmaf(f.x, LOG2E, -mL));
                s += ex2_ftz(fmaf(f.y, LOG2E, -mL));
            }
        }
    }
    if (has_tail) s += ex2_ftz(fmaf(tv, LOG2E, -mL));
    s = block_reduce(s, false, red);
    const float inv_s = __fdiv_rn(1.0f, s);
    const float k = inv_s * c;
    if (tid == 0) row_loss[row] = (m + (logf(s) - delta * 0.69314718055994531f)) - hbits2f(zr[y]);

#pragma unroll
    for (int u = 0; u < VPT; u++) {
        const int i = tid + u * nt;
        if (i < C8) {
            const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; q++) {
                const float2 f = __half22float2(*(const __half2 *)&w[q]);
                const __half2 h = __floats2half2_rn(ex2_ftz(fmaf(f.x, LOG2E, -mL)) * k, ex2_ftz(fmaf(f.y, LOG2E, -mL)) * k);
                o[q] = *(const uint32_t *)&h;
            }
            __stcs((uint4 *)dr + i, make_uint4(o[0], o[1], o[2], o[3]));
        }
    }
    if (has_tail) dr[C8 * 8 + tid] = (uint16_t)f2hbits(ex2_ftz(fmaf(tv, LOG2E, -mL)) * k);
    __syncthreads();  // the row's stores are done before the label element is patched
    if (tid == 0) {
        const float ey = ex2_ftz(fmaf(hbits2f(zr[y]), LOG2E, -mL));
        dr[y] = (uint16_t)f2hbits(__fmul_rn(__fsub_rn(ey * inv_s, 1.0f), c));
    }
}


// ---------------------------------------------------------------- rows staged by bulk copies
//
// Persistent form for rows whose bytes are a multiple of 16 and fit three times into shared
// memory: one CTA per SM walks rows blockIdx.x, blockIdx.x + gridDim.x, ...  A row arrives by one
// bulk asynchronous copy (cp.async.bulk, completion on an mbarrier), is turned into its gradient in
// place, and leaves by one bulk store; with three row buffers the load of row k+1 and the store of
// row k-1 are in flight while the threads work on row k, so the memory system always has work.
// Arithmetic as in k_softmax_ce_reg.  The waits are bounded like those of the product kernels.
static constexpr int kSmaxThreads = 1024;

// Block-wide max or sum for exactly 32 warps: warp results go through shared memory, then every
// warp combines the 32 of them with the same xor-butterfly (both partners of a step add the same
// two numbers, so all lanes and all warps hold identical bits; the order is fixed).
// any_out (may be null): receives the OR of `pred` over the block, carried by the reduction's barrier.
__device__ __forceinline__ float block_reduce32(float v, bool is_max, float *red, bool pred = false, int *any_out = nullptr)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = is_max ? fmaxf(v, other) : v + other;
    }
    if (lane == 0) red[warp] = v;   // the caller alternates between two arrays: no reuse hazard
    if (any_out) *any_out = __syncthreads_or(pred ? 1 : 0);
    else __syncthreads();
    float r = red[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xFFFFFFFFu, r, o);
        r = is_max ? fmaxf(r, other) : r + other;
    }
    return r;
}

__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    mbar_arrive_expect_tx(bar, bytes);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store_row(void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <int VPT>
__global__ void __launch_bounds__(kSmaxThreads, 1) k_softmax_ce_bulk(const uint16_t *__restrict__ z, int ldz,
                                                                      const int32_t *__restrict__ labels, int B, int C, float c,
                                                                      uint16_t *__restrict__ dz, int lddz,
                                                                      float *__restrict__ row_loss, uint32_t *bad_labels,
                                                                      const float *__restrict__ scale_dev, uint32_t *kerr)
{
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(128) uint8_t rows_smem[];
    __shared__ float red[2][32];   // max and sum use different arrays; a row's last use is two barriers back
    __shared__ __align__(8) uint64_t bars[3];
    __shared__ uint32_t abort_word;
    if (scale_dev) c = __fdiv_rn(*scale_dev, (float)B);
    const int tid = threadIdx.x;
    const uint32_t row_bytes = (uint32_t)C * 2u;
    const uint32_t buf_stride = (row_bytes + 127u) & ~127u;
    const int C8 = C >> 3;
    if (tid == 0) {
        for (int i = 0; i < 3; i++) mbar_init(smem_u32(&bars[i]), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int n_my = blockIdx.x < B ? (B - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const uint32_t smem0 = smem_u32(rows_smem);
    if (tid == 0 && n_my > 0) bulk_load_row(smem0, z + (size_t)blockIdx.x * ldz, row_bytes, smem_u32(&bars[0]));
    constexpr float LOG2E = 1.4426950408889634f;
    for (int k = 0; k < n_my; k++) {
        const int row = blockIdx.x + k * gridDim.x;
        const int b = k % 3;
        if (tid == 0 && k + 1 < n_my) {
            // buffer (k+1)%3 last held row k-2: its store must have finished reading shared memory
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            bulk_load_row(smem0 + (uint32_t)((k + 1) % 3) * buf_stride, z + (size_t)(row + gridDim.x) * ldz, row_bytes,
                          smem_u32(&bars[(k + 1) % 3]));
        }
        // every thread waits for the row itself; whether any of them gave up is learnt on the barrier
        // of the first reduction (a thread that gave up scans stale data until then, harmlessly)
        const bool arrived = mbar_wait(smem_u32(&bars[b]), (uint32_t)((k / 3) & 1), &abort_word);
        if (!arrived) abort_word = 1;
        uint4 *rowv = (uint4 *)(rows_smem + (size_t)b * buf_stride);
        uint16_t *rowh = (uint16_t *)rowv;
        const int y = labels[row];
        const bool good = y >= 0 && y < C;
        // the thread that will write the vector holding the label's element also patches it
        const bool owner = good && tid == ((y >> 3) & (kSmaxThreads - 1));
        float zy = 0.0f;
        if (owner) zy = hbits2f(rowh[y]);                  // read long before the row is overwritten in place
        // pass 1: the maximum, on packed FP16 values (max is exact in any precision; like fmaxf it
        // drops NaN operands, which then surface through the exponentials)
        __half2 mh = __half2half2(__ushort_as_half((unsigned short)0xFC00u));   // -inf
#pragma unroll
        for (int u = 0; u < VPT; u++) {
            const int i = tid + u * kSmaxThreads;
            if (i < C8) {
                const uint4 x = rowv[i];
                mh = __hmax2(mh, __hmax2(__hmax2(*(const __half2 *)&x.x, *(const __half2 *)&x.y),
                                         __hmax2(*(const __half2 *)&x.z, *(const __half2 *)&x.w)));
            }
        }
        float m = fmaxf(__low2float(mh), __high2float(mh));
        int gave_up = 0;
        m = block_reduce32(m, true, red[0], !arrived, &gave_up);
        if (gave_up) {
            if (kerr && tid == 0) atomicCAS(kerr, 0u, (uint32_t)KERR_WAIT_FULL | 0x40u | ((uint32_t)blockIdx.x << 8));
            break;
        }
        // pass 2: exponentials, kept in registers for pass 3, and their sum.  One FMA and one
        // special-function instruction per logit: 2^(z*log2e - mL) with mL = rn(m*log2e).  Rounding mL
        // scales every exponential of the row by the same 2^delta (delta = m*log2e - mL, obtained
        // exactly by an FMA): it cancels in e/s and is taken out of log(s) below.
        const float mL = __fmul_rn(m, LOG2E);
        const float delta = fmaf(m, LOG2E, -mL);
        float ev[VPT * 8];
        float s = 0.0f;
#pragma unroll
        for (int u = 0; u < VPT; u++) {
            const int i = tid + u * kSmaxThreads;
            if (i < C8) {
                const uint4 x = rowv[i];
                const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    const float2 f = __half22float2(*(const __half2 *)&w[q]);
                    ev[u * 8 + 2 * q] = ex2_ftz(fmaf(f.x, LOG2E, -mL));
                    ev[u * 8 + 2 * q + 1] = ex2_ftz(fmaf(f.y, LOG2E, -mL));
                    s += ev[u * 8 + 2 * q];
                    s += ev[u * 8 + 2 * q + 1];
                }
            }
        }
        s = block_reduce32(s, false, red[1]);
        const float inv_s = __fdiv_rn(1.0f, s);
        const float kk = inv_s * c;
        if (good) {
#pragma unroll
            for (int u = 0; u < VPT; u++) {
                const int i = tid + u * kSmaxThreads;
                if (i < C8) {
                    uint32_t o[4];
#pragma unroll
                    for (int q = 0; q < 4; q++) {
                        const __half2 h = __floats2half2_rn(ev[u * 8 + 2 * q] * kk, ev[u * 8 + 2 * q + 1] * kk);
                        o[q] = *(const uint32_t *)&h;
                    }
                    rowv[i] = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
        } else {           // a label outside [0, C): the whole gradient row is zero
#pragma unroll
            for (int u = 0; u < VPT; u++) {
                const int i = tid + u * kSmaxThreads;
                if (i < C8) rowv[i] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        // the label's element: d_y = (e_y / s - 1) * c, evaluated separately because of the
        // cancellation; its owner wrote the vector around it just above, so no block barrier is needed
        // (the warp-level one keeps the two stores, made through different pointer types, in order)
        __syncwarp();
        if (owner) {
            const float ey = ex2_ftz(fmaf(zy, LOG2E, -mL));
            rowh[y] = (uint16_t)f2hbits(__fmul_rn(__fsub_rn(ey * inv_s, 1.0f), c));
            row_loss[row] = (m + (logf(s) - delta * 0.69314718055994531f)) - zy;
        } else if (!good && tid == 0) {   // a label outside [0, C) contributes neither loss nor gradient
            row_loss[row] = 0.0f;
            if (bad_labels) atomicAdd(bad_labels, 1u);
        }
        // every thread's shared-memory writes become visible to the bulk store
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) bulk_store_row(dz + (size_t)row * lddz, smem0 + (uint32_t)b * buf_stride, row_bytes);
    }
    if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}



// loss = (float)( sum_i (double)row_loss[i] / B ), fixed reduction order.
__global__ void __launch_bounds__(256) k_loss_mean(const float *__restrict__ row_loss, int B, float *loss)
{
    pdl_trigger();
    pdl_wait();
    __shared__ double red[256];
    double acc = 0.0;
    for (int i = threadIdx.x; i < B; i += 256) acc += (double)row_loss[i];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = (B > 0) ? (float)(red[0] / (double)B) : 0.0f;
}

template <bool VEC, bool CACHE>
static cudaError_t launch_variant(const uint16_t *z, int ldz, const int32_t *labels, int B, int C, float c,
                                  uint16_t *dz, int lddz, float *row_loss, uint32_t *bad_labels, int threads,
                                  int grid, size_t smem, cudaStream_t st, const float *S_dev)
{
    auto kern = k_softmax_ce<VEC, CACHE>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    MPT_LAUNCH(kern, dim3(grid), dim3(threads), smem, st, z, ldz, labels, B, C, c, dz, lddz, row_loss, bad_labels, S_dev);
    return cudaGetLastError();
}

cudaError_t launch_softmax_ce(const uint16_t *z, int ldz, const int32_t *labels, int B, int C, float S,
                              uint16_t *dz, int lddz, float *row_loss, float *loss, uint32_t *bad_labels,
                              cudaStream_t st, int *n_launches, const float *S_dev, uint32_t *kerr)
{
    if (n_launches) *n_launches = 0;
    if (B <= 0 || C <= 0) return cudaSuccess;
    const float c = S / (float)B;  // one FP32 division
    const bool vec = ((((uintptr_t)z | (uintptr_t)dz) & 15) == 0) && (ldz % 8 == 0) && (lddz % 8 == 0) && C >= 8;
    // many long rows: persistent CTAs with rows staged through shared memory by bulk copies
    if (vec && (C % 8) == 0 && C >= 16384 && C <= 32768 && B >= 2 * 148) {
        static int sms_dev[kMaxDevices] = {};
        const int dev = current_device_slot();
        if (dev < 0) return cudaErrorInvalidDevice;
        const size_t smem = 3 * (((size_t)C * 2 + 127) & ~(size_t)127);
        const int vpt = (C >> 3) <= 2048 ? 2 : 4;
        auto kern = vpt == 2 ? k_softmax_ce_bulk<2> : k_softmax_ce_bulk<4>;
        if (sms_dev[dev] == 0) {
            int n = 0;
            cudaError_t e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return e;
            e = cudaFuncSetAttribute(k_softmax_ce_bulk<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(k_softmax_ce_bulk<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e != cudaSuccess) return e;
            sms_dev[dev] = n > 0 ? n : 148;
        }
        const int grid = B < sms_dev[dev] ? B : sms_dev[dev];
        MPT_LAUNCH(kern, dim3(grid), dim3(kSmaxThreads), smem, st, z, ldz, labels, B, C, c, dz, lddz, row_loss, bad_labels, S_dev, kerr);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (n_launches) *n_launches = 1;
        if (loss) {
            MPT_LAUNCH(k_loss_mean, dim3(1), dim3(256), 0, st, row_loss, B, loss);
            if (n_launches) *n_launches = 2;
        }
        return cudaGetLastError();
    }
    if (vec && (C >> 3) <= 8 * 1024) {
        // register-resident rows: T threads x VPT vectors cover C / 8 vectors
        const int C8 = C >> 3;
        int vpt = 1;
        while (vpt < 8 && (long)vpt * 1024 < C8) vpt *= 2;
        int threads = (C8 + vpt - 1) / vpt;
        threads = ((threads + 31) / 32) * 32;
        if (threads < 32) threads = 32;
        switch (vpt) {
            case 1: MPT_LAUNCH(k_softmax_ce_reg<1>, dim3(B), dim3(threads), 0, st, z, ldz, labels, C, c, dz, lddz, row_loss, bad_labels, S_dev); break;
            case 2: MPT_LAUNCH(k_softmax_ce_reg<2>, dim3(B), dim3(threads), 0, st, z, ldz, labels, C, c, dz, lddz, row_loss, bad_labels, S_dev); break;
            case 4: MPT_LAUNCH(k_softmax_ce_reg<4>, dim3(B), dim3(threads), 0, st, z, ldz, labels, C, c, dz, lddz, row_loss, bad_labels, S_dev); break;
            default: MPT_LAUNCH(k_softmax_ce_reg<8>, dim3(B), dim3(threads), 0, st, z, ldz, labels, C, c, dz, lddz, row_loss, bad_labels, S_dev); break;
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (n_launches) *n_launches = 1;
        if (loss) {
            MPT_LAUNCH(k_loss_mean, dim3(1), dim3(256), 0, st, row_loss, B, loss);
            if (n_launches) *n_launches = 2;
        }
        return cudaGetLastError();
    }
    const size_t row_bytes = ((size_t)C * 2 + 15) & ~(size_t)15;
    const bool cache = row_bytes <= (size_t)kMaxSmemRowBytes;
    int threads = vec ? (C / 8) : C;
    threads = ((threads + 31) / 32) * 32;
    if (threads > 1024) threads = 1024;
    if (threads < 32) threads = 32;
    int grid = B < 148 * 16 ? B : 148 * 16;
    size_t smem = cache ? row_bytes : 0;
    cudaError_t e;
    if (vec && cache) e = launch_variant<true, true>(z, ldz, labels, B, C, c, dz, lddz, row_loss, bad_labels, threads, grid, smem, st, S_dev);
    else if (vec) e = launch_variant<true, false>(z, ldz, labels, B, C, c, dz, lddz, row_loss, bad_labels, threads, grid, smem, st, S_dev);
    else if (cache) e = launch_variant<false, true>(z, ldz, labels, B, C, c, dz, lddz, row_loss, bad_labels, threads, grid, smem, st, S_dev);
    else e = launch_variant<false, false>(z, ldz, labels, B, C, c, dz, lddz, row_loss, bad_labels, threads, grid, smem, st, S_dev);
    if (e != cudaSuccess) return e;
    if (n_launches) *n_launches = 1;
    if (loss) {
        MPT_LAUNCH(k_loss_mean, dim3(1), dim3(256), 0, st, row_loss, B, loss);
        if (n_launches) *n_launches = 2;
    }
    return cudaGetLastError();
}

}  // namespace mpt

// ---------------------------------------------------------------------------------
// Variant of mpt_softmax_ce whose per-row loss scratch lives inside the library.
//
// The array below is part of the loaded module: every GPU that loads this library
// holds these 256 KiB from load until the process exits, and every call on that GPU
// shares them.  In host code the name g_static_row_loss is only a handle for the
// symbol, not an address a kernel can use; the device address is obtained once per
// device with cudaGetSymbolAddress while that device is current, and that pointer
// is what the kernels receive.
static __device__ __align__(256) float g_static_row_loss[MPT_SOFTMAX_STATIC_MAX_ROWS];

namespace {
float *g_static_ptr[mpt::kMaxDevices];   // per device, filled on the first call made with that device current
}  // namespace

extern "C" int mpt_softmax_ce_static(const uint16_t *z_dev, int ldz, const int32_t *labels_dev, int B, int C, float S,
                                     uint16_t *dz_dev, int lddz, float *loss_dev, uint32_t *bad_labels_dev,
                                     uint32_t *status_dev, void *cuda_stream)
{
    if (!z_dev || !labels_dev || !dz_dev || !loss_dev) return MPT_ERR_INVALID_ARG;
    if (B < 0 || C < 0 || ldz < C || lddz < C) return MPT_ERR_SHAPE;
    if (B > MPT_SOFTMAX_STATIC_MAX_ROWS) return MPT_ERR_SHAPE;   // the built-in scratch holds one float per row
    if (z_dev == dz_dev) return MPT_ERR_INVALID_ARG;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return MPT_ERR_CUDA;
    if (device < 0 || device >= mpt::kMaxDevices) return MPT_ERR_INTERNAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // The array's address belongs to the CURRENT device; a stream of another device would hand its
    // kernels a pointer into the wrong GPU's copy of the array.
    int stream_device = device;
    if (cudaStreamGetDevice(st, &stream_device) != cudaSuccess) return MPT_ERR_CUDA;
    if (stream_device != device) return MPT_ERR_INVALID_ARG;
    if (!g_static_ptr[device]) {
        float *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_static_row_loss) != cudaSuccess || !p) return MPT_ERR_CUDA;
        g_static_ptr[device] = p;
    }
    cudaError_t e = cudaSuccess;
    if (bad_labels_dev) e = cudaMemsetAsync(bad_labels_dev, 0, sizeof(uint32_t), st);
    // Nothing in the scratch has to start at zero: rows 0..B-1 are each written by the row
    // kernel before the mean kernel reads exactly those rows; older contents are never read.
    if (e == cudaSuccess)
        e = mpt::launch_softmax_ce(z_dev, ldz, labels_dev, B, C, S, dz_dev, lddz, g_static_ptr[device], loss_dev,
                                   bad_labels_dev, st, nullptr, nullptr, status_dev);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

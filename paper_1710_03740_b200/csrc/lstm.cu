// LSTM layer pieces outside the tensor-core products (sections 3.3, 4.5 of the paper): the
// backward of the gate arithmetic, the FP32 bias-gradient reduction, the FP16 add of two
// gradient contributions, and a plain-CUDA-core forward cell for shapes the tensor-core
// kernels do not take.  All of them are memory-bound streaming kernels on FP16 storage with
// FP32 arithmetic; every FP32 operation is rounded separately, in the order the header documents.
#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

namespace {

__device__ __forceinline__ float h2f_u(uint32_t h) { return __half2float(__ushort_as_half((unsigned short)h)); }
__device__ __forceinline__ uint32_t f2h_u(float x) { return (uint32_t)__half_as_ushort(__float2half_rn(x)); }

// ------------------------------------------------------------ forward cell, CUDA cores

// One thread per (row, cell): four dot products in ascending k with FP32 accumulation, then the
// same gate arithmetic as the fused tensor-core epilogue.  For small or unaligned shapes only.
__global__ void __launch_bounds__(256) k_lstm_cell_simt(int B, int H, int K, const uint16_t *__restrict__ XR, int ldxr,
                                                        const uint16_t *__restrict__ Wg, int ldw,
                                                        uint16_t *__restrict__ acts, int ldacts, LstmEpi e)
{
    pdl_trigger();
    pdl_wait();
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)B * H) return;
    const int b = (int)(idx / H), j = (int)(idx % H);
    const uint16_t *x = XR + (size_t)b * ldxr;
    float pre[4];
#pragma unroll
    for (int q = 0; q < 4; q++) {
        const uint16_t *w = Wg + (size_t)(4 * j + q) * ldw;
        float acc = 0.0f;
        for (int k = 0; k < K; k++) acc = __fadd_rn(acc, __fmul_rn(h2f_u(x[k]), h2f_u(w[k])));
        pre[q] = __fadd_rn(acc, h2f_u(e.bias[4 * j + q]));
    }
    uint32_t act[4], c16, h16;
    lstm_cell_math(pre, h2f_u(e.c_prev[(size_t)b * e.ldcp + j]), act, c16, h16);
#pragma unroll
    for (int q = 0; q < 4; q++) acts[(size_t)b * ldacts + 4 * j + q] = (uint16_t)act[q];
    e.c_out[(size_t)b * e.ldco + j] = (uint16_t)c16;
    e.h_out[(size_t)b * e.ldh + j] = (uint16_t)h16;
}

// ------------------------------------------------------------ backward of the gate arithmetic

struct CellGrad {
    uint32_t dg[4];   // FP16 bits of the gradients wrt the four pre-activations
    uint32_t dcp;     // FP16 bits of the gradient wrt c_{t-1}
};

__device__ __forceinline__ CellGrad cell_bwd(float gi, float gf, float gg, float go, float cp, float c, float dh, float dcn)
{
    const float tc = tanhf(c);   // accurate: 1 - tc*tc below cancels, so an approximate tanh would show in dc
    const float dc = __fadd_rn(__fmul_rn(__fmul_rn(dh, go), __fsub_rn(1.0f, __fmul_rn(tc, tc))), dcn);
    const float dpo = __fmul_rn(__fmul_rn(dh, tc), __fmul_rn(go, __fsub_rn(1.0f, go)));
    const float dpi = __fmul_rn(__fmul_rn(dc, gg), __fmul_rn(gi, __fsub_rn(1.0f, gi)));
    const float dpf = __fmul_rn(__fmul_rn(dc, cp), __fmul_rn(gf, __fsub_rn(1.0f, gf)));
    const float dpg = __fmul_rn(__fmul_rn(dc, gi), __fsub_rn(1.0f, __fmul_rn(gg, gg)));
    CellGrad r;
    r.dg[0] = f2h_u(dpi); r.dg[1] = f2h_u(dpf); r.dg[2] = f2h_u(dpg); r.dg[3] = f2h_u(dpo);
    r.dcp = f2h_u(__fmul_rn(dc, gf));
    return r;
}

// Four cells per thread: two 128-bit loads of the activations, 64-bit loads of the per-cell values
// (streaming hints: nothing is read twice).  H is a multiple of 4 and all pitches are multiples of 4
// (checked by the launcher), so the 64-bit accesses are aligned.
__global__ void __launch_bounds__(256) k_lstm_cell_bwd(int B, int H4, const uint16_t *__restrict__ dh, int lddh,
                                                       const uint16_t *__restrict__ dc_next, int lddc,
                                                       const uint16_t *__restrict__ acts, int ldacts,
                                                       const uint16_t *__restrict__ c_prev, int ldcp,
                                                       const uint16_t *__restrict__ c16, int ldc, uint16_t *__restrict__ dG,
                                                       int lddg, uint16_t *__restrict__ dc_prev, int lddcp)
{
    pdl_trigger();
    pdl_wait();
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)B * H4) return;
    const int b = (int)(idx / H4), j = 4 * (int)(idx % H4);
    const uint4 *ap = (const uint4 *)(acts + (size_t)b * ldacts + 4 * j);
    const uint4 a0 = __ldcs(ap), a1 = __ldcs(ap + 1);
    const uint2 cpw = __ldcs((const uint2 *)(c_prev + (size_t)b * ldcp + j));
    const uint2 cw = __ldcs((const uint2 *)(c16 + (size_t)b * ldc + j));
    const uint2 dhw = __ldcs((const uint2 *)(dh + (size_t)b * lddh + j));
    const uint2 dcw = dc_next ? __ldcs((const uint2 *)(dc_next + (size_t)b * lddc + j)) : make_uint2(0u, 0u);
    const uint32_t aw[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    const uint32_t cp2[2] = {cpw.x, cpw.y}, c2[2] = {cw.x, cw.y}, dh2[2] = {dhw.x, dhw.y}, dc2[2] = {dcw.x, dcw.y};
    uint32_t outg[8], outc[2];
#pragma unroll
    for (int k = 0; k < 4; k++) {
        const int sh = (k & 1) * 16;
        const CellGrad g = cell_bwd(h2f_u(aw[2 * k] & 0xFFFFu), h2f_u(aw[2 * k] >> 16), h2f_u(aw[2 * k + 1] & 0xFFFFu),
                                    h2f_u(aw[2 * k + 1] >> 16), h2f_u((cp2[k >> 1] >> sh) & 0xFFFFu),
                                    h2f_u((c2[k >> 1] >> sh) & 0xFFFFu), h2f_u((dh2[k >> 1] >> sh) & 0xFFFFu),
                                    h2f_u((dc2[k >> 1] >> sh) & 0xFFFFu));
        outg[2 * k] = g.dg[0] | (g.dg[1] << 16);
        outg[2 * k + 1] = g.dg[2] | (g.dg[3] << 16);
        if (k & 1) outc[k >> 1] |= g.dcp << 16;
        else outc[k >> 1] = g.dcp;
    }
    uint4 *gp = (uint4 *)(dG + (size_t)b * lddg + 4 * j);
    __stcs(gp, make_uint4(outg[0], outg[1], outg[2], outg[3]));
    __stcs(gp + 1, make_uint4(outg[4], outg[5], outg[6], outg[7]));
    __stcs((uint2 *)(dc_prev + (size_t)b * lddcp + j), make_uint2(outc[0], outc[1]));
}

// scalar form for odd H or unaligned buffers
__global__ void __launch_bounds__(256) k_lstm_cell_bwd_scalar(int B, int H, const uint16_t *__restrict__ dh, int lddh,
                                                              const uint16_t *__restrict__ dc_next, int lddc,
                                                              const uint16_t *__restrict__ acts, int ldacts,
                                                              const uint16_t *__restrict__ c_prev, int ldcp,
                                                              const uint16_t *__restrict__ c16, int ldc,
                                                              uint16_t *__restrict__ dG, int lddg,
                                                              uint16_t *__restrict__ dc_prev, int lddcp)
{
    pdl_trigger();
    pdl_wait();
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)B * H) return;
    const int b = (int)(idx / H), j = (int)(idx % H);
    const uint16_t *a = acts + (size_t)b * ldacts + 4 * j;
    const CellGrad g = cell_bwd(h2f_u(a[0]), h2f_u(a[1]), h2f_u(a[2]), h2f_u(a[3]), h2f_u(c_prev[(size_t)b * ldcp + j]),
                                h2f_u(c16[(size_t)b * ldc + j]), h2f_u(dh[(size_t)b * lddh + j]),
                                dc_next ? h2f_u(dc_next[(size_t)b * lddc + j]) : 0.0f);
    uint16_t *d = dG + (size_t)b * lddg + 4 * j;
    d[0] = (uint16_t)g.dg[0]; d[1] = (uint16_t)g.dg[1]; d[2] = (uint16_t)g.dg[2]; d[3] = (uint16_t)g.dg[3];
    dc_prev[(size_t)b * lddcp + j] = (uint16_t)g.dcp;
}

// ------------------------------------------------------------ bias gradient

// Column sums in FP32 (section 3.3: reductions in FP32).  Fixed partition: the rows are cut into
// kBiasRowParts contiguous ranges (blockIdx.y); inside a CTA warp w takes rows w, w+8, ... of
// its range in ascending order, lane l the 8 columns 8l..8l+7 of the CTA's 256-column block; the
// eight warps are combined in ascending order through shared memory into parts[range][column].
__global__ void __launch_bounds__(256) k_bias_grad_partial(const uint16_t *__restrict__ dG, size_t rows, int cols, int ld,
                                                           float *__restrict__ parts, bool vec)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float sh[8][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col = blockIdx.x * 256 + lane * 8;
    const size_t per = (rows + gridDim.y - 1) / gridDim.y;
    const size_t r0 = (size_t)blockIdx.y * per;
    const size_t r1 = r0 + per < rows ? r0 + per : rows;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (vec && col + 8 <= cols) {
        for (size_t r = r0 + warp; r < r1; r += 8) {
            const uint4 v = __ldcs((const uint4 *)(dG + r * (size_t)ld + col));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 8; e++)
                acc[e] = __fadd_rn(acc[e], h2f_u((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu)));
        }
    } else {
        for (size_t r = r0 + warp; r < r1; r += 8)
            for (int e = 0; e < 8 && col + e < cols; e++) acc[e] = __fadd_rn(acc[e], h2f_u(dG[r * (size_t)ld + col + e]));
    }
#pragma unroll
    for (int e = 0; e < 8; e++) sh[warp][lane * 8 + e] = acc[e];
    __syncthreads();
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c < cols) {
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; w++) s = __fadd_rn(s, sh[w][threadIdx.x]);
        parts[(size_t)blockIdx.y * cols + c] = s;
    }
}

__global__ void __launch_bounds__(256) k_bias_grad_final(const float *__restrict__ parts, int nparts, int cols,
                                                         uint16_t *__restrict__ db16, uint32_t *nonfinite_flag)
{
    pdl_trigger();
    pdl_wait();
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    bool bad = false;
    if (c < cols) {
        float s = 0.0f;
        for (int p = 0; p < nparts; p++) s = __fadd_rn(s, parts[(size_t)p * cols + c]);
        const uint32_t h = f2h_u(s);
        bad = half_bits_nonfinite(h);
        db16[c] = (uint16_t)h;
    }
    if (nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && (threadIdx.x & 31) == 0) atomicOr(nonfinite_flag, 1u);
}

// ------------------------------------------------------------ FP16 add

__global__ void __launch_bounds__(256) k_add_f16(const uint16_t *__restrict__ a, int lda, const uint16_t *__restrict__ b,
                                                 int ldb, uint16_t *__restrict__ out, int ldo, int rows, int cols)
{
    pdl_trigger();
    pdl_wait();
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)rows * cols) return;
    const int r = (int)(idx / cols), c = (int)(idx % cols);
    out[(size_t)r * ldo + c] = (uint16_t)f2h_u(__fadd_rn(h2f_u(a[(size_t)r * lda + c]), h2f_u(b[(size_t)r * ldb + c])));
}

__global__ void __launch_bounds__(256) k_widen_f16(const uint16_t *__restrict__ in16, float *__restrict__ out32, size_t n)
{
    pdl_trigger();
    pdl_wait();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out32[i] = h2f_u(in16[i]);
}

unsigned blocks_for(size_t n) { return (unsigned)((n + 255) / 256); }

}  // namespace

cudaError_t launch_lstm_cell_simt(int B, int H, int K, const uint16_t *XR, int ldxr, const uint16_t *Wg, int ldw,
                                  uint16_t *acts, int ldacts, const LstmEpi &e, cudaStream_t st)
{
    if (B <= 0 || H <= 0) return cudaSuccess;
    MPT_LAUNCH(k_lstm_cell_simt, dim3(blocks_for((size_t)B * H)), dim3(256), 0, st, B, H, K, XR, ldxr, Wg, ldw, acts, ldacts, e);
    return cudaGetLastError();
}

cudaError_t launch_lstm_cell_bwd(int B, int H, const uint16_t *dh, int lddh, const uint16_t *dc_next, int lddc,
                                 const uint16_t *acts, int ldacts, const uint16_t *c_prev, int ldcp, const uint16_t *c16,
                                 int ldc, uint16_t *dG, int lddg, uint16_t *dc_prev, int lddcp, cudaStream_t st)
{
    if (B <= 0 || H <= 0) return cudaSuccess;
    const uintptr_t bits = (uintptr_t)acts | (uintptr_t)dG;
    const uintptr_t bits4 = (uintptr_t)dh | (uintptr_t)dc_next | (uintptr_t)c_prev | (uintptr_t)c16 | (uintptr_t)dc_prev;
    const bool vec = (H % 4) == 0 && (bits & 15) == 0 && (bits4 & 7) == 0 && (ldacts % 8) == 0 && (lddg % 8) == 0 &&
                     ((lddh | lddc | ldcp | ldc | lddcp) % 4) == 0;
    if (vec)
        MPT_LAUNCH(k_lstm_cell_bwd, dim3(blocks_for((size_t)B * (H / 4))), dim3(256), 0, st, B, H / 4, dh, lddh, dc_next, lddc, acts, ldacts, c_prev,
                   ldcp, c16, ldc, dG, lddg, dc_prev, lddcp);
    else
        MPT_LAUNCH(k_lstm_cell_bwd_scalar, dim3(blocks_for((size_t)B * H)), dim3(256), 0, st, B, H, dh, lddh, dc_next, lddc, acts, ldacts, c_prev,
                   ldcp, c16, ldc, dG, lddg, dc_prev, lddcp);
    return cudaGetLastError();
}

cudaError_t launch_bias_grad(const uint16_t *dG, size_t rows, int cols, int ld, float *parts, uint16_t *db16,
                             uint32_t *nonfinite_flag, cudaStream_t st)
{
    if (cols <= 0) return cudaSuccess;
    const bool vec = ((uintptr_t)dG & 15) == 0 && (ld % 8) == 0;
    dim3 grid((unsigned)((cols + 255) / 256), (unsigned)kBiasRowParts);
    MPT_LAUNCH(k_bias_grad_partial, dim3(grid), dim3(256), 0, st, dG, rows, cols, ld, parts, vec);   // unaligned rows: element loads
    MPT_LAUNCH(k_bias_grad_final, dim3(blocks_for((size_t)cols)), dim3(256), 0, st, parts, kBiasRowParts, cols, db16, nonfinite_flag);
    return cudaGetLastError();
}

cudaError_t launch_widen_f16(const uint16_t *in16, float *out32, size_t n, cudaStream_t st)
{
    if (n == 0) return cudaSuccess;
    MPT_LAUNCH(k_widen_f16, dim3(blocks_for(n)), dim3(256), 0, st, in16, out32, n);
    return cudaGetLastError();
}

cudaError_t launch_add_f16(const uint16_t *a, int lda, const uint16_t *b, int ldb, uint16_t *out, int ldo, int rows,
                           int cols, cudaStream_t st)
{
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    MPT_LAUNCH(k_add_f16, dim3(blocks_for((size_t)rows * cols)), dim3(256), 0, st, a, lda, b, ldb, out, ldo, rows, cols);
    return cudaGetLastError();
}

}  // namespace mpt

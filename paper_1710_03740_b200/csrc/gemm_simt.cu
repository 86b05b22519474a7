// CUDA-core FP16 GEMM with FP32 accumulation (paper section 3.3), used for operands
// the tensor-core kernel cannot take (unaligned pitches, e.g. 10 logits) and as an
// on-device cross-check.  Every output sums its products for k = 0..K-1 in ascending
// order with one FP32 rounding per term (the product of two FP16 values is exact in
// FP32, so the fused multiply-add below rounds exactly like multiply-then-add).
#include "mpt_common.cuh"

namespace mpt {

static constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;

__device__ __forceinline__ float ldh(const uint16_t *p) { return __half2float(__ushort_as_half(*p)); }

// C[m,n] = sum_k A(m,k) B(k,n);  A(m,k) = ATRANS ? A[k*lda+m] : A[m*lda+k];
//                                 B(k,n) = BTRANS ? B[k*ldb+n] : B[n*ldb+k].
template <bool ATRANS, bool BTRANS>
__global__ void __launch_bounds__(256) k_gemm_simt(int M, int N, int K, const uint16_t *__restrict__ A, int lda,
                                                   const uint16_t *__restrict__ B, int ldb, uint16_t *__restrict__ C,
                                                   int ldc, int relu, const uint16_t *__restrict__ mask, int ldmask,
                                                   uint32_t *nonfinite_flag)
{
    pdl_trigger();
    pdl_wait();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; i++)
#pragma unroll
        for (int j = 0; j < TN; j++) acc[i][j] = 0.0f;

    for (int k0 = 0; k0 < K; k0 += BK) {
        // stage a BK x BM slab of A and a BK x BN slab of B as FP32 (4 elements per thread each)
#pragma unroll
        for (int r = 0; r < 4; r++) {
            int kk, mm;
            if (ATRANS) { kk = tid / 64 + 4 * r; mm = tid % 64; }
            else        { kk = tid % 16;         mm = tid / 16 + 16 * r; }
            int gk = k0 + kk, gm = m0 + mm;
            float v = 0.0f;
            if (gk < K && gm < M) v = ATRANS ? ldh(A + (size_t)gk * lda + gm) : ldh(A + (size_t)gm * lda + gk);
            As[kk][mm] = v;
            int nn;
            if (BTRANS) { kk = tid / 64 + 4 * r; nn = tid % 64; }
            else        { kk = tid % 16;         nn = tid / 16 + 16 * r; }
            gk = k0 + kk;
            int gn = n0 + nn;
            v = 0.0f;
            if (gk < K && gn < N) v = BTRANS ? ldh(B + (size_t)gk * ldb + gn) : ldh(B + (size_t)gn * ldb + gk);
            Bs[kk][nn] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; kk++) {   // ascending k; zero padding adds exact zeros
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; i++) a[i] = As[kk][ty * TM + i];
#pragma unroll
            for (int j = 0; j < TN; j++) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
            for (int i = 0; i < TM; i++)
#pragma unroll
                for (int j = 0; j < TN; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

    bool bad = false;
#pragma unroll
    for (int i = 0; i < TM; i++) {
        int gm = m0 + ty * TM + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < TN; j++) {
            int gn = n0 + tx * TN + j;
            if (gn >= N) continue;
            float s = acc[i][j];
            if (relu) s = (s > 0.0f) ? s : ((s != s) ? s : 0.0f);
            uint16_t h = __half_as_ushort(__float2half_rn(s));
            if (mask && !(ldh(mask + (size_t)gm * ldmask + gn) > 0.0f)) h = 0;
            bad |= half_bits_nonfinite(h);
            C[(size_t)gm * ldc + gn] = h;
        }
    }
    if (nonfinite_flag && __any_sync(0xFFFFFFFFu, bad) && (tid & 31) == 0) atomicOr(nonfinite_flag, 1u);
}

cudaError_t launch_gemm_simt(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                             uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask,
                             uint32_t *nonfinite_flag, cudaStream_t st)
{
    if (M <= 0 || N <= 0) return cudaSuccess;
    dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM);
    if (op == MPT_OP_FWD)
        MPT_LAUNCH(k_gemm_simt<false, false>, dim3(grid), dim3(256), 0, st, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag);
    else if (op == MPT_OP_DGRAD)
        MPT_LAUNCH(k_gemm_simt<false, true>, dim3(grid), dim3(256), 0, st, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag);
    else
        MPT_LAUNCH(k_gemm_simt<true, true>, dim3(grid), dim3(256), 0, st, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag);
    return cudaGetLastError();
}

}  // namespace mpt

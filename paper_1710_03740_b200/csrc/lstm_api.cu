// C entry points of the LSTM layer (see mpt.h): argument checks and the launch sequence over time
// steps.  Every arithmetic step runs in a kernel; the host only orders launches on one stream.
#include <stdint.h>

#include "mpt_common.cuh"

using namespace mpt;

namespace {

bool valid_desc(const mpt_lstm_desc *d)
{
    if (!d) return false;
    if (d->T < 1 || d->B < 1 || d->I < 8 || d->H < 8 || d->P < 8) return false;
    if ((d->I % 8) || (d->H % 8) || (d->P % 8)) return false;
    if ((long long)d->H * 4 > 0x7FFFFFF0ll || (long long)d->T * d->B > 0x7FFFFFF0ll) return false;
    return true;
}

// gate product + gate arithmetic of one step: tensor-core kernel with the fused epilogue when the
// shapes allow, CUDA-core cell otherwise
int cell_forward(int B, int H, int K, const uint16_t *xr, int ldxr, const uint16_t *Wg, int ldw, uint16_t *acts, int ldacts,
                 const LstmEpi &e, unsigned flags, uint32_t *status_dev, cudaStream_t st)
{
    const int N = 4 * H;
    const bool aligned = (N % 32) == 0 && (e.ldcp % 8) == 0 && (e.ldco % 8) == 0 && (e.ldh % 8) == 0 &&
                         (((uintptr_t)e.bias | (uintptr_t)e.c_prev | (uintptr_t)e.c_out | (uintptr_t)e.h_out) & 15) == 0;
    const bool tc_ok = aligned && K > 0 && tc_gemm_supported(MPT_OP_FWD, B, N, K, xr, ldxr, Wg, ldw, acts, ldacts, nullptr, 0);
    if ((flags & (MPT_GEMM_FORCE_TC | MPT_GEMM_FORCE_PAIR)) && !tc_ok) return MPT_ERR_SHAPE;
    if (tc_ok && !(flags & MPT_GEMM_FORCE_SIMT))
        return dispatch_gemm(MPT_OP_FWD, B, N, K, xr, ldxr, Wg, ldw, acts, ldacts, flags, nullptr, 0, nullptr, status_dev, nullptr,
                             0, st, &e);
    return launch_lstm_cell_simt(B, H, K, xr, ldxr, Wg, ldw, acts, ldacts, e, st) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

}  // namespace

extern "C" {

int mpt_lstm_cell_forward(int B, int H, int K, const uint16_t *xr, int ldxr, const uint16_t *Wg, int ldw,
                          const uint16_t *bias16, const uint16_t *c_prev, int ldcp, uint16_t *acts, int ldacts,
                          uint16_t *c_out, int ldco, uint16_t *h_out, int ldh, unsigned flags, uint32_t *status_dev,
                          void *cuda_stream)
{
    if (!xr || !Wg || !bias16 || !c_prev || !acts || !c_out || !h_out) return MPT_ERR_INVALID_ARG;
    if (B < 0 || H < 0 || K < 0) return MPT_ERR_SHAPE;
    if (B == 0 || H == 0) return MPT_OK;
    if (ldxr < K || ldw < K || ldacts < 4 * H || ldcp < H || ldco < H || ldh < H) return MPT_ERR_SHAPE;
    LstmEpi e{bias16, nullptr, c_prev, ldcp, c_out, ldco, h_out, ldh};
    return cell_forward(B, H, K, xr, ldxr, Wg, ldw, acts, ldacts, e, flags, status_dev, (cudaStream_t)cuda_stream);
}

int mpt_lstm_cell_backward(int B, int H, const uint16_t *dh, int lddh, const uint16_t *dc_next, int lddc,
                           const uint16_t *acts, int ldacts, const uint16_t *c_prev, int ldcp, const uint16_t *c16, int ldc,
                           uint16_t *dG, int lddg, uint16_t *dc_prev, int lddcp, void *cuda_stream)
{
    if (!dh || !acts || !c_prev || !c16 || !dG || !dc_prev) return MPT_ERR_INVALID_ARG;
    if (B < 0 || H < 0) return MPT_ERR_SHAPE;
    if (lddh < H || (dc_next && lddc < H) || ldacts < 4 * H || ldcp < H || ldc < H || lddg < 4 * H || lddcp < H)
        return MPT_ERR_SHAPE;
    return launch_lstm_cell_bwd(B, H, dh, lddh, dc_next, lddc, acts, ldacts, c_prev, ldcp, c16, ldc, dG, lddg, dc_prev, lddcp,
                                (cudaStream_t)cuda_stream) == cudaSuccess
               ? MPT_OK
               : MPT_ERR_CUDA;
}

int mpt_bias_grad(const uint16_t *dG, size_t rows, int cols, int ld, float *parts, uint16_t *db16, uint32_t *nonfinite_flag,
                  void *cuda_stream)
{
    if (!dG || !parts || !db16) return MPT_ERR_INVALID_ARG;
    if (cols < 0 || ld < cols) return MPT_ERR_SHAPE;
    return launch_bias_grad(dG, rows, cols, ld, parts, db16, nonfinite_flag, (cudaStream_t)cuda_stream) == cudaSuccess
               ? MPT_OK
               : MPT_ERR_CUDA;
}

int mpt_add_f16(const uint16_t *a, int lda, const uint16_t *b, int ldb, uint16_t *out, int ldo, int rows, int cols,
                void *cuda_stream)
{
    if (!a || !b || !out) return MPT_ERR_INVALID_ARG;
    if (rows < 0 || cols < 0 || lda < cols || ldb < cols || ldo < cols) return MPT_ERR_SHAPE;
    return launch_add_f16(a, lda, b, ldb, out, ldo, rows, cols, (cudaStream_t)cuda_stream) == cudaSuccess ? MPT_OK
                                                                                                          : MPT_ERR_CUDA;
}

int mpt_lstm_forward(const mpt_lstm_desc *d, const mpt_lstm_tensors *t, void *cuda_stream)
{
    if (!d || !t) return MPT_ERR_INVALID_ARG;
    if (!valid_desc(d)) return MPT_ERR_SHAPE;
    if (!t->Wg16 || !t->bias16 || !t->Wp16 || !t->xr || !t->c || !t->h || !t->acts) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int B = d->B, I = d->I, H = d->H, P = d->P, K = I + P;
    const size_t xr_step = (size_t)B * K, c_step = (size_t)B * H, a_step = (size_t)B * 4 * H;
    // the first 4H floats of the bias-gradient scratch hold an exact FP32 copy of the bias during
    // the forward pass: the gate epilogue then needs no FP16->FP32 conversions for it
    const float *bias32 = nullptr;
    if (t->bias_parts && (((uintptr_t)t->bias_parts) & 15) == 0) {
        if (launch_widen_f16(t->bias16, t->bias_parts, (size_t)4 * H, st) != cudaSuccess) return MPT_ERR_CUDA;
        bias32 = t->bias_parts;
    }
    for (int s = 0; s < d->T; s++) {
        LstmEpi e{t->bias16, bias32, t->c + s * c_step, H, t->c + (s + 1) * c_step, H, t->h + s * c_step, H};
        int r = cell_forward(B, H, K, t->xr + s * xr_step, K, t->Wg16, K, t->acts + s * a_step, 4 * H, e, 0, t->status_dev, st);
        if (r != MPT_OK) return r;
        // r_s = h_s . Wp^T, written into the recurrent columns of the next step's input rows
        r = dispatch_gemm(MPT_OP_FWD, B, P, H, t->h + s * c_step, H, t->Wp16, H, t->xr + (s + 1) * xr_step + I, K, 0, nullptr, 0,
                          nullptr, t->status_dev, t->splitk_ws, t->splitk_ws ? t->splitk_ws_bytes : 0, st, nullptr);
        if (r != MPT_OK) return r;
    }
    return MPT_OK;
}

int mpt_lstm_backward(const mpt_lstm_desc *d, const mpt_lstm_tensors *t, void *cuda_stream)
{
    if (!d || !t) return MPT_ERR_INVALID_ARG;
    if (!valid_desc(d)) return MPT_ERR_SHAPE;
    if (!t->Wg16 || !t->Wp16 || !t->xr || !t->c || !t->h || !t->acts || !t->dr_ext || !t->dxr || !t->drtot || !t->dG || !t->dh ||
        !t->dc || !t->dWg16 || !t->dWp16 || !t->dbias16 || !t->bias_parts)
        return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int T = d->T, B = d->B, I = d->I, H = d->H, P = d->P, K = I + P;
    const size_t xr_step = (size_t)B * K, c_step = (size_t)B * H, a_step = (size_t)B * 4 * H, p_step = (size_t)B * P;
    for (int s = T - 1; s >= 0; s--) {
        uint16_t *drtot = t->drtot + s * p_step;
        cudaError_t ce;
        if (s == T - 1)
            ce = cudaMemcpyAsync(drtot, t->dr_ext + s * p_step, p_step * 2, cudaMemcpyDeviceToDevice, st);
        else
            ce = launch_add_f16(t->dr_ext + s * p_step, P, t->dxr + (s + 1) * xr_step + I, K, drtot, P, B, P, st);
        if (ce != cudaSuccess) return MPT_ERR_CUDA;
        // dh_s = drtot_s . Wp
        int r = dispatch_gemm(MPT_OP_DGRAD, B, H, P, drtot, P, t->Wp16, H, t->dh, H, 0, nullptr, 0, nullptr, t->status_dev, nullptr, 0,
                              st, nullptr);
        if (r != MPT_OK) return r;
        uint16_t *dc_out = t->dc + (size_t)(s & 1) * c_step;
        const uint16_t *dc_in = s == T - 1 ? nullptr : t->dc + (size_t)((s + 1) & 1) * c_step;
        ce = launch_lstm_cell_bwd(B, H, t->dh, H, dc_in, H, t->acts + s * a_step, 4 * H, t->c + s * c_step, H,
                                  t->c + (s + 1) * c_step, H, t->dG + s * a_step, 4 * H, dc_out, H, st);
        if (ce != cudaSuccess) return MPT_ERR_CUDA;
        // dxr_s = dG_s . Wg
        r = dispatch_gemm(MPT_OP_DGRAD, B, K, 4 * H, t->dG + s * a_step, 4 * H, t->Wg16, K, t->dxr + s * xr_step, K, 0, nullptr, 0,
                          nullptr, t->status_dev, nullptr, 0, st, nullptr);
        if (r != MPT_OK) return r;
    }
    // weight gradients over all T*B rows: the sum over time is accumulated in FP32 inside the product
    const int rows = T * B;
    int r = dispatch_gemm(MPT_OP_WGRAD, 4 * H, K, rows, t->dG, 4 * H, t->xr, K, t->dWg16, K, 0, nullptr, 0, t->nonfinite_flag,
                          t->status_dev, nullptr, 0, st, nullptr);
    if (r != MPT_OK) return r;
    r = dispatch_gemm(MPT_OP_WGRAD, P, H, rows, t->drtot, P, t->h, H, t->dWp16, H, 0, nullptr, 0, t->nonfinite_flag, t->status_dev,
                      nullptr, 0, st, nullptr);
    if (r != MPT_OK) return r;
    if (launch_bias_grad(t->dG, (size_t)rows, 4 * H, 4 * H, t->bias_parts, t->dbias16, t->nonfinite_flag, st) != cudaSuccess)
        return MPT_ERR_CUDA;
    return MPT_OK;
}

}  // extern "C"

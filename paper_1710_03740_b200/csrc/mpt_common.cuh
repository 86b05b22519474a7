// Shared declarations of the CUDA library: kernel launcher prototypes and small
// device helpers.  Internal; the public boundary is include/mpt.h.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mpt.h"

namespace mpt {

// Device status block (uint32 words) inside a context's workspace.
enum StatusWord : int {
    ST_OVERFLOW = 0,      // OR of "weight gradient is inf/NaN" (wgrad epilogues, detect kernel)
    ST_OVERFLOW_SEEN = 1, // the update kernel's own inspection of the gradients it streamed
    ST_BAD_LABELS = 2,    // labels outside [0, C) seen by the last softmax
    ST_KERNEL_ERR = 3,    // first device-side error (bounded wait expired): code | where<<8
    ST_LOSS = 4,          // float: unscaled mean loss of the last backward
    ST_SCALE = 5,         // float: loss scale S the next backward / master pass will use
    ST_INV_SCALE = 6,     // float: 1.0f / S (one FP32 division)
    ST_CLEAN_STEPS = 7,   // consecutive steps without overflow since S last changed (dynamic scaling)
    ST_B1T = 8,           // float: beta1^t over the applied (not skipped) steps (Adam)
    ST_B2T = 9,           // float: beta2^t
    ST_CLIP_COEF = 10,    // float: clipping coefficient of the last step (global-norm clipping)
    ST_GRAD_NORM = 11,    // float: norm of the unscaled gradients of the last step
    ST_DP_NORM = 12,      // double (words 12, 13): this replica's shard of the squared norm of the mean gradient
    ST_WORDS = 16
};

// Device-side error codes written to ST_KERNEL_ERR.
enum KernelErr : uint32_t {
    KERR_NONE = 0,
    KERR_WAIT_FULL = 1,   // consumer gave up waiting for a TMA-filled stage
    KERR_WAIT_EMPTY = 2,  // producer gave up waiting for a free stage
    KERR_WAIT_ACC = 3,    // epilogue gave up waiting for the accumulator
    KERR_WAIT_ACC_FREE = 4, // MMA issuer gave up waiting for a drained accumulator
    KERR_TMEM_ALLOC = 5,
    KERR_WAIT_SELFTEST = 6, // the self-test's wait on a barrier nobody signals ran out, as intended
    KERR_WAIT_PARTIAL = 7   // a warp gave up waiting for another CTA pair's part of a split contraction
};

// Kernel attributes (opt-in shared memory size, cluster occupancy) are per device: launchers
// keep one "configured" slot per device ordinal.
static constexpr int kMaxDevices = 64;
inline int current_device_slot()
{
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) return -1;
    return d;
}

// Programmatic dependent launch.  Every kernel of the library starts with pdl_trigger() (its
// dependents may be scheduled as soon as all of its CTAs have started) and executes pdl_wait()
// before its first access to global memory (the wait returns when the preceding kernel in the
// stream has completed and its writes are visible).  What runs before the wait - barrier set-up,
// tensor-memory allocation, the launch itself - overlaps the tail of the preceding kernel.  In a
// kernel launched without the attribute both are no-ops.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with programmatic stream serialization (see above); kernels launched this way must call
// pdl_wait() before touching global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Launch through launch_pdl and return its error from the calling function if the launch failed.
#define MPT_LAUNCH(...)                                      \
    do {                                                     \
        cudaError_t launch_err_ = launch_pdl(__VA_ARGS__);   \
        if (launch_err_ != cudaSuccess) return launch_err_;  \
    } while (0)

__device__ __forceinline__ bool half_bits_nonfinite(uint32_t h) { return (h & 0x7C00u) == 0x7C00u; }
__device__ __forceinline__ bool f32_nonfinite(float x)
{
    return (__float_as_uint(x) & 0x7F800000u) == 0x7F800000u;
}

// Fused LSTM gate epilogue of a forward product whose output columns are gate-interleaved
// (column 4j+q = gate q of cell j; q: 0 input, 1 forget, 2 candidate, 3 output): the FP32
// accumulators plus bias go through the gate non-linearities, the product's own output receives
// the FP16 gate activations, and the new cell state and hidden state are written beside it.
// All pitches are multiples of 8 elements and all bases 16-byte aligned.
struct LstmEpi {
    const uint16_t *bias;     // [4H] FP16 working copy
    const float *bias32;      // [4H] the same values converted to FP32 (exactly), or null
    const uint16_t *c_prev;   // [B, H], pitch ldcp
    int ldcp;
    uint16_t *c_out;          // [B, H], pitch ldco
    int ldco;
    uint16_t *h_out;          // [B, H], pitch ldh
    int ldh;
};

// Launchers (each returns a cudaError_t from the launch; all asynchronous on `st`).
cudaError_t launch_recast(const float *w32, uint16_t *w16, size_t n, cudaStream_t st);
cudaError_t launch_grad_nonfinite(const uint16_t *g16, size_t n, float inv_S, uint32_t *flag,
                                  cudaStream_t st);
// inv_S_dev / S_dev (may be null): when given, the kernel reads 1/S resp. S from device memory
// instead of taking the by-value argument (the scale can then change without a host round trip).
cudaError_t launch_update(const uint16_t *g16, float *w32, float *v, uint16_t *w16, size_t n, float inv_S,
                          float lr, float mu, bool use_momentum, uint32_t *flags, cudaStream_t st,
                          const float *inv_S_dev = nullptr);
cudaError_t launch_softmax_ce(const uint16_t *z, int ldz, const int32_t *labels, int B, int C, float S,
                              uint16_t *dz, int lddz, float *row_loss, float *loss, uint32_t *bad_labels,
                              cudaStream_t st, int *n_launches, const float *S_dev = nullptr, uint32_t *kerr = nullptr);
// One warp measures its SM's clock over window_us of wall time and writes MHz to *mhz_out (clock_probe.cu).
cudaError_t launch_clock_probe(unsigned window_us, float *mhz_out, cudaStream_t st);
// One CTA waits, for at most limit_us, on a barrier nothing arrives on; on expiry it records
// KERR_WAIT_SELFTEST in *status (wait_selftest.cu).
cudaError_t launch_wait_selftest(unsigned limit_us, uint32_t *status, cudaStream_t st);
// Optimizer steps other than SGD(+momentum), and weight decay (see mpt.h MPT_OPT_*).  s1 / s2:
// FP32 state arrays (momentum or squared-gradient sum; Adam's second moment).  For Adam the
// bias corrections are 1 - beta^t with beta^t either passed by value (b1t, b2t: the products
// INCLUDING this step) or, when betat_dev is given, read as the products of the previous applied
// steps from device memory and multiplied by beta once more in the kernel.
cudaError_t launch_update_opt(int kind, const uint16_t *g16, float *w32, float *s1, float *s2, uint16_t *w16, size_t n,
                              float inv_S, float lr, float mu, float b2, float eps, float wd, float b1t, float b2t,
                              uint32_t *flags, cudaStream_t st, const float *inv_S_dev, const float *betat_dev,
                              const float *coef_dev = nullptr);
// Global-norm clipping of the unscaled gradients: a fixed-partition double-precision sum of
// squares over g16[0..n) into parts[kNormParts], then out2[0] = min(1, clip/(norm + 1e-6)) and
// out2[1] = norm as FP32.  launch_update_opt multiplies every unscaled gradient by *coef_dev.
static constexpr int kNormParts = 1184;
cudaError_t launch_clip_coef(const uint16_t *g16, size_t n, float inv_S, const float *inv_S_dev, float clip, double *parts,
                             float *out2, cudaStream_t st);
// Data-parallel step for one replica's shard (see mpt.h, mpt_dp_step_flat): g16 / flag / w16 are
// host arrays of R device pointers; w32_shard / v_shard point at element `first` of the owner's
// state, `count` elements.  S_dev (may be null): the loss scale is read from device memory and
// 1/(S*R) formed in the kernel (one multiplication, one division) instead of taking inv_SR.
cudaError_t launch_dp_step(const uint16_t *const *g16, const uint32_t *const *flag, uint16_t *const *w16, int R,
                           float *w32_shard, float *v_shard, size_t first, size_t count, float inv_SR, const float *S_dev,
                           float lr, float mu, uint32_t *flags, cudaStream_t st, int *n_launches);
// The same with the optimizer steps of launch_update_opt on the mean gradient (no clipping).
cudaError_t launch_dp_step_opt(int kind, const uint16_t *const *g16, const uint32_t *const *flag, uint16_t *const *w16, int R,
                               float *w32_shard, float *s1_shard, float *s2_shard, size_t first, size_t count, float inv_SR,
                               const float *S_dev, float lr, float mu, float b2, float eps, float wd, float b1t, float b2t,
                               const float *betat_dev, uint32_t *flags, cudaStream_t st, int *n_launches,
                               const float *coef_dev = nullptr, const float *sum32 = nullptr);
// The FP32 sums over the replicas of elements [first, first + count) of their gradient arrays (multiples of
// 8), stored at sum32_out[0 .. count); launch_dp_step_opt takes them through its sum32 argument (indexed
// like w32_shard) in place of the gradients.
cudaError_t launch_dp_reduce(const uint16_t *const *g16, int R, size_t first, size_t count, float *sum32_out, cudaStream_t st);
// Clipping in the data-parallel step: this replica's shard of the sum of squares of the mean unscaled
// gradient (double) into *slot (parts: scratch of kDpNormScratch doubles); then, once every replica
// has published its slot, out2[0] = coefficient, out2[1] = norm from all R slots in replica order.
static constexpr int kDpNormScratch = 592;
cudaError_t launch_dp_sqnorm(const uint16_t *const *g16, int R, size_t first, size_t count, float inv_SR, const float *S_dev,
                             double *parts, double *slot, cudaStream_t st, const float *sum32 = nullptr);
cudaError_t launch_dp_clip_coef(const double *const *slots, int R, float clip, float *out2, cudaStream_t st);
// End-of-step bookkeeping on the device (one thread): dynamic loss scale (if interval > 0) and
// Adam's running products beta^t (if adam != 0); both only move on a step that was applied.
cudaError_t launch_post_step(uint32_t *status, int interval, float backoff, float growth, float min_S, float max_S,
                             int adam, float b1, float b2, cudaStream_t st);

// Dynamic loss scaling (one thread): on overflow S <- max(S * backoff, min_S) and the clean-step
// counter restarts; after `interval` clean steps S <- min(S * growth, max_S).  Rewrites the
// ST_SCALE / ST_INV_SCALE / ST_CLEAN_STEPS words of the status block.
cudaError_t launch_scale_adjust(uint32_t *status, int interval, float backoff, float growth, float min_S,
                                float max_S, cudaStream_t st);
cudaError_t launch_gemm_simt(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B,
                             int ldb, uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask,
                             uint32_t *nonfinite_flag, cudaStream_t st);

// tcgen05 path.  tc_gemm_supported: alignment/shape rules; launch_gemm_tc builds the
// TMA descriptors on the host and launches the persistent kernel.
bool tc_gemm_supported(int op, int M, int N, int K, const void *A, int lda, const void *B, int ldb,
                       const void *C, int ldc, const void *mask, int ldmask);
// splitk_ws (may be null): 16-byte aligned device scratch for split-K partial sums; without it
// the contraction is never split.  tc_gemm_plan tells which tile width / split factor the
// launcher will pick and how much scratch that needs.
cudaError_t launch_gemm_tc(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B,
                           int ldb, uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask,
                           uint32_t *nonfinite_flag, uint32_t *status, cudaStream_t st, float *splitk_ws = nullptr,
                           size_t splitk_ws_bytes = 0, const LstmEpi *lstm = nullptr);
void tc_gemm_plan(int M, int N, int K, size_t ws_bytes, int *bn_out, int *split_out, size_t *ws_needed,
                  double *cost_out = nullptr);
// Kernel choice for a product the tensor-core path takes: true = CTA-pair kernel (possibly with a
// split contraction), false = single-CTA kernel; ws_needed = scratch the choice would like.
bool tc_choose_pair(int M, int N, int K, size_t ws_bytes, size_t *ws_needed);

// Number of kernels the last product launcher called on this host thread enqueued (the product
// kernel plus, for a split contraction or a split tail, the reduce kernel): bookkeeping only.
extern thread_local int g_last_gemm_launches;

// CTA-pair variant (tcgen05 cta_group::2, 256x256 tiles); same operand rules as launch_gemm_tc.
bool tc2_gemm_preferred(int M, int N, int K);
cudaError_t launch_gemm_tc2(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                            uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask,
                            uint32_t *nonfinite_flag, uint32_t *status, cudaStream_t st, const LstmEpi *lstm = nullptr,
                            void *splitk_ws = nullptr, size_t splitk_ws_bytes = 0);
// Second step of a split product: C = epilogue(partial[0] + partial[1] + ...), parts added in
// ascending order with one rounding per add.
cudaError_t launch_splitk_reduce(const float *partial, int split_k, int M, int N, int ldp, uint16_t *C, int ldc, bool relu,
                                 const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag, cudaStream_t st);
// CTA-pair variant with 256x512 tiles (two accumulators fed by one stream of A; the epilogue is
// not overlapped): less operand traffic, not faster; only on request (MPT_GEMM_FORCE_PAIR512).
cudaError_t launch_gemm_tc3(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                            uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask,
                            uint32_t *nonfinite_flag, uint32_t *status, cudaStream_t st);
// In-cluster split (gemm_tc4.cu): a cluster of `split` CTA pairs (2 or 4) per 256x256 tile, each pair
// running 1/split of the contraction, parts added through distributed shared memory; no scratch, one
// launch.  tc4_split_for: the split this kernel would use for a shape, 0 when it is not the kernel for it.
int tc4_split_for(int M, int N, int K);
cudaError_t launch_gemm_tc4(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb,
                            uint16_t *C, int ldc, bool relu, const uint16_t *mask, int ldmask,
                            uint32_t *nonfinite_flag, uint32_t *status, cudaStream_t st, int split);
size_t tc2_tail_ws_bytes(int M, int N, int K);
// Split factor, scratch need (FP32 parts) and modelled cost
// of the pair kernel for an output with few tiles and a long contraction; split 1 = no split.
void tc2_split_plan(int M, int N, int K, size_t ws_bytes, int *split_out, size_t *ws_needed, double *cost_out);

// Shape checks and kernel choice for one product (used by the stateless entry points and the LSTM
// layer); returns an MPT_* code.
int dispatch_gemm(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb, uint16_t *C, int ldc,
                  unsigned flags, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag, uint32_t *status_dev,
                  void *splitk_ws_dev, size_t splitk_ws_bytes, cudaStream_t st, const LstmEpi *lstm);

// LSTM layer pieces outside the products (see mpt.h, mpt_lstm_*):
// gate product + gate arithmetic for shapes the tensor-core kernels do not take (any size, slow)
cudaError_t launch_lstm_cell_simt(int B, int H, int K, const uint16_t *XR, int ldxr, const uint16_t *Wg, int ldw,
                                  uint16_t *acts, int ldacts, const LstmEpi &e, cudaStream_t st);
// backward of the gate arithmetic of one time step (dc_next may be null: zero)
cudaError_t launch_lstm_cell_bwd(int B, int H, const uint16_t *dh, int lddh, const uint16_t *dc_next, int lddc,
                                 const uint16_t *acts, int ldacts, const uint16_t *c_prev, int ldcp, const uint16_t *c16,
                                 int ldc, uint16_t *dG, int lddg, uint16_t *dc_prev, int lddcp, cudaStream_t st);
// db16[n] = rn16(sum over rows of dG[r, n]) with FP32 accumulation over a fixed partition;
// parts: FP32 scratch [kBiasRowParts][cols]
static constexpr int kBiasRowParts = 8;
cudaError_t launch_bias_grad(const uint16_t *dG, size_t rows, int cols, int ld, float *parts, uint16_t *db16,
                             uint32_t *nonfinite_flag, cudaStream_t st);
// out32[i] = f32(in16[i]) (exact)
cudaError_t launch_widen_f16(const uint16_t *in16, float *out32, size_t n, cudaStream_t st);
// out = rn16(f32(a) + f32(b)) over a [rows, cols] block with pitches
cudaError_t launch_add_f16(const uint16_t *a, int lda, const uint16_t *b, int ldb, uint16_t *out, int ldo, int rows,
                           int cols, cudaStream_t st);

}  // namespace mpt

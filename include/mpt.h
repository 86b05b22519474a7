/*
 * mpt.h -- C ABI of the B200 (sm_100a) mixed-precision training hot path.
 *
 * The library implements one training iteration of a stack of bias-free linear
 * layers in the recipe of "Mixed Precision Training" (arXiv 1710.03740):
 *
 *   section 3.1  weights, activations and gradients are stored as FP16; an FP32
 *                master copy of the weights receives the update and is rounded
 *                to the FP16 working copy used by forward and backward;
 *   section 3.2  the loss is multiplied by a constant S before back-propagation;
 *                weight gradients are multiplied by 1/S before the update and
 *                inspected for inf/NaN, in which case the update is skipped;
 *   section 3.3  dot products take FP16 operands, accumulate in FP32 and convert
 *                to FP16 on the store; softmax reductions run in FP32 on FP16
 *                data; point-wise ops (ReLU) are fused into the producers.
 *
 * Conventions
 *   - Every tensor is row-major, last index contiguous.  FP16 values cross this
 *     boundary as uint16_t bit patterns (IEEE binary16).  Rounding FP32 -> FP16
 *     is round-to-nearest-even with gradual underflow everywhere.
 *   - "_dev" pointers are CUDA device pointers, "_host" pointers are host
 *     pointers (pageable or pinned).  Nothing in a signature is a torch type.
 *   - The model-level calls (mpt_create ... mpt_destroy) and the stateless launchers never
 *     allocate or free device memory and never create a stream.  The caller owns the
 *     workspace, the inputs, the stream and all host buffers; the library owns only its
 *     host-side context object.  Exceptions, each documented at its declaration:
 *     mpt_dp_alloc / mpt_dp_free obtain and release device memory from the driver;
 *     mpt_dp_overlap_events / mpt_dp_overlap_attach create events and one more stream, which
 *     mpt_destroy releases;
 *     mpt_softmax_ce_static uses a fixed device array inside the library that all calls on a
 *     GPU share; and the launchers keep small per-device host-side caches that are filled on
 *     first use (SM count, opt-in shared-memory sizes, cluster occupancy, the address of that
 *     array).  Because of those caches the FIRST call of each kernel on a device makes CUDA
 *     runtime queries and must come before any stream capture.
 *   - Every call returns MPT_OK (0) or a negative MPT_ERR_* code and never
 *     throws.  A null context or a null required pointer gives
 *     MPT_ERR_INVALID_ARG with nothing dereferenced.  Calls are asynchronous on
 *     the context's stream unless a host out-pointer is passed, in which case
 *     the call synchronises the stream before writing it.
 *   - After MPT_ERR_CUDA or MPT_ERR_TIMEOUT the context is poisoned: only
 *     mpt_last_error and mpt_destroy succeed.
 *   - A context is not thread-safe; distinct contexts are independent.
 */
#ifndef MPT_H_
#define MPT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MPT_OK 0
#define MPT_ERR_INVALID_ARG (-1) /* null pointer, bad enum, bad scalar */
#define MPT_ERR_SHAPE (-2)       /* dimensions inconsistent or out of range */
#define MPT_ERR_STATE (-3)       /* call order violated (e.g. backward before forward) */
#define MPT_ERR_WORKSPACE (-4)   /* workspace too small or misaligned */
#define MPT_ERR_CUDA (-5)        /* a CUDA runtime/driver call failed */
#define MPT_ERR_TIMEOUT (-6)     /* a bounded device-side wait expired */
#define MPT_ERR_INTERNAL (-7)    /* internal consistency check failed */

/* Which index of the stored operands is contracted (section 3.3; the three
 * products of one layer's iteration, section 3.1):
 *   FWD    C[M,N] = A[M,K] . B[N,K]^T     Y  = X  W^T
 *   DGRAD  C[M,N] = A[M,K] . B[K,N]       dX = dY W
 *   WGRAD  C[M,N] = A[K,M]^T . B[K,N]     dW = dY^T X                      */
#define MPT_OP_FWD 0
#define MPT_OP_DGRAD 1
#define MPT_OP_WGRAD 2

/* mpt_gemm_f16 flags */
#define MPT_GEMM_RELU 1u      /* apply x > 0 ? x : +0 to the FP32 sum before rounding */
#define MPT_GEMM_FORCE_SIMT 2u /* use the plain CUDA-core kernel (sequential-k FP32 sum) */
#define MPT_GEMM_FORCE_TC 4u   /* require the single-CTA tcgen05 kernel (128x256 tiles);
                                  MPT_ERR_SHAPE if the operands do not meet its alignment rules */
#define MPT_GEMM_FORCE_PAIR 8u /* require the CTA-pair tcgen05 kernel (cta_group::2, 256x256 tiles);
                                  same alignment rules.  Without a FORCE flag the library picks the
                                  pair kernel when the output has more 256x256 tiles than the 74 CTA
                                  pairs run at once (or at least 48 with K >= 16384), the in-cluster
                                  split for few tiles and a long K (below), else the single-CTA one */
#define MPT_GEMM_FORCE_PAIR512 16u /* require the CTA-pair kernel with 256x512 tiles (two accumulators
                                  fed by one stream of A, epilogue not overlapped); same alignment
                                  rules.  Moves about a quarter fewer operand bytes and is not faster;
                                  never picked automatically */
#define MPT_GEMM_FORCE_SPLIT2 32u /* require the in-cluster split kernel: a cluster of two CTA pairs per
                                  256x256 tile, each pair running half of the contraction, the two FP32
                                  accumulators added through distributed shared memory (parts in ascending
                                  order, one rounding per add) before the one rounding to FP16.  Same
                                  alignment rules; K >= 128.  Picked automatically for outputs of at most
                                  32 tiles with K >= 2048 (section 4.5's projection product) */
#define MPT_GEMM_FORCE_SPLIT4 64u /* the same with four CTA pairs per tile (a cluster of eight CTAs), each
                                  running a quarter of the contraction; K >= 256.  Picked automatically
                                  for outputs of at most 12 tiles with K >= 4096 */

/* mpt_get_tensor kinds */
#define MPT_T_W16 0        /* FP16 working weights   [out, in]            */
#define MPT_T_GRAD16 1     /* FP16 weight gradients  [out, in] (scaled by S) */
#define MPT_T_ACT16 2      /* FP16 activation a_l    [batch, out_l]       */
#define MPT_T_DACT16 3     /* FP16 gradient dz_l     [batch, out_l] (scaled by S) */
#define MPT_T_MOMENTUM32 4 /* FP32 momentum buffer   [out, in]            */
#define MPT_T_MASTER32 5   /* FP32 master weights    [out, in]            */
#define MPT_T_STATE2_32 6  /* FP32 second optimizer state [out, in] (Adam's second moment) */

/* Optimizer step applied to the FP32 master copy (section 3.1: the update is computed in FP32;
 * the paper's experiments use plain and Nesterov momentum SGD, Adagrad and Adam, sections 4.3,
 * 4.5, 4.6, without giving formulas: the textbook forms are used).  With g the UNSCALED
 * gradient (section 3.2: clipping, decay and the like act after unscaling), every line one
 * separately rounded FP32 operation, states starting at zero:
 *   clip_norm > 0:      g = g * coef, coef = min(1, clip_norm / (norm + 1e-6)) rounded to FP32,
 *                       norm = sqrt(sum over ALL layers of g*g), sum, sqrt and quotient in double
 *                       (one extra read of the FP16 gradients: +2 bytes per parameter)
 *   weight_decay != 0:  g = g + weight_decay * w
 *   MPT_OPT_SGD       momentum == 0: u = lr*g ;  else  s1 = momentum*s1 + g ; u = lr*s1
 *   MPT_OPT_NESTEROV  s1 = momentum*s1 + g ; u = lr*(g + momentum*s1)
 *   MPT_OPT_ADAGRAD   s1 = s1 + g*g ; u = lr*(g / (sqrt(s1) + eps))
 *   MPT_OPT_ADAM      s1 = b1*s1 + (1-b1)*g ; s2 = b2*s2 + (1-b2)*(g*g) ;
 *                     u = lr*((s1/(1-b1^t)) / (sqrt(s2/(1-b2^t)) + eps))   (b1 = momentum field)
 *                     where b^t are running FP32 products over the steps that were applied
 *                     (a step skipped for overflow does not advance them)
 *   w = w - u ; w16 = rn16(w)
 * Bytes moved per parameter: 12 (plain SGD), 20 (one state), 28 (Adam). */
#define MPT_OPT_SGD 0
#define MPT_OPT_NESTEROV 1
#define MPT_OPT_ADAGRAD 2
#define MPT_OPT_ADAM 3

typedef struct mpt_optimizer {
    int32_t kind;       /* MPT_OPT_* */
    float lr;
    float momentum;     /* SGD / Nesterov momentum, Adam beta1; in [0, 1) */
    float beta2;        /* Adam beta2 in [0, 1); ignored otherwise */
    float eps;          /* Adagrad / Adam epsilon >= 0; ignored otherwise */
    float weight_decay; /* >= 0; 0 disables */
    float clip_norm;    /* >= 0; bound on the global norm of the unscaled gradients; 0 disables */
} mpt_optimizer;

typedef struct mpt_ctx mpt_ctx;

typedef struct mpt_layer_desc {
    int32_t in_features;
    int32_t out_features;
    int32_t relu; /* 1: ReLU after this layer (hidden layers); the last layer must be 0 */
} mpt_layer_desc;

/* ------------------------------------------------------------ model-level calls */

/* Size in bytes of the single device workspace a context needs (section 3.1:
 * FP32 master + FP16 weights + FP16 gradients, optional FP32 momentum, FP16
 * activations and activation gradients for max_batch rows, two input staging
 * slots, per-row losses and status words).  Host-only; no CUDA call. */
int mpt_workspace_bytes(const mpt_layer_desc *layers, int n_layers, int max_batch,
                        int use_momentum, size_t *bytes_out);

/* Create a context over a caller-allocated workspace (section 3.1, 3.2: the
 * iteration's state: master weights, loss scale S, learning rate).
 *   layers/n_layers  chain of linear layers, out_l == in_{l+1}, last layer relu == 0
 *   S                constant loss scale, finite, 2^-100 <= S <= 2^120
 *   lr               learning rate, finite
 *   momentum         0 <= momentum < 1; 0 selects plain SGD (no momentum buffer)
 *   max_batch        largest batch later passed to mpt_forward
 *   workspace_dev    device memory, 256-byte aligned, >= mpt_workspace_bytes(...)
 *   cuda_stream      a cudaStream_t (may be 0 for the default stream); all work
 *                    of this context is issued on it
 * Zeroes the momentum and gradient buffers.  Master weights are undefined until
 * mpt_set_master has been called for every layer. */
int mpt_create(const mpt_layer_desc *layers, int n_layers, float S, float lr, float momentum,
               int max_batch, void *workspace_dev, size_t workspace_bytes, void *cuda_stream,
               mpt_ctx **out);

/* mpt_workspace_bytes / mpt_create for any optimizer of the list above (mpt_create is the SGD
 * case: kind MPT_OPT_SGD with the given lr and momentum). */
int mpt_workspace_bytes_opt(const mpt_layer_desc *layers, int n_layers, int max_batch, const mpt_optimizer *opt,
                            size_t *bytes_out);
int mpt_create_opt(const mpt_layer_desc *layers, int n_layers, float S, const mpt_optimizer *opt, int max_batch,
                   void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out);

/* Upload one layer's FP32 master weights [out, in] from the host and round them
 * to the FP16 working copy (section 3.1).  n must equal out*in.  Synchronous. */
int mpt_set_master(mpt_ctx *ctx, int layer, const float *src_host, size_t n);

/* Forward pass (section 3.3): for l = 1..L
 *   a_l[i,j] = rn16( act( sum_k a_{l-1}[i,k] * w16_l[j,k] ) ), sum in FP32.
 * x_dev: FP16 [batch, in_1] with row pitch in_1, read-only, caller-owned; it must
 * stay valid and unchanged until the stream work of the following
 * mpt_backward_scaled has completed (the first layer's weight gradient reads it).
 * 1 <= batch <= max_batch.  The logits are a_L (MPT_T_ACT16, layer L-1). */
int mpt_forward(mpt_ctx *ctx, const uint16_t *x_dev, int batch);

/* Scaled backward pass (sections 3.2, 3.3).  Softmax cross-entropy over the
 * logits in FP32: loss = mean_i (logsumexp(z_i) - z_i[y_i]), logit gradient
 * dz_L = rn16((softmax(z_i) - onehot(y_i)) * S / batch); then for l = L..1
 *   gW_l[j,k]   = rn16( sum_i dz_l[i,j] * a_{l-1}[i,k] )
 *   dz_{l-1}[i,k] = [a_{l-1}[i,k] > 0] * rn16( sum_j dz_l[i,j] * w16_l[j,k] )  (l > 1)
 * The gradient buffers are overwritten, not accumulated into.
 * labels_dev: int32 [batch] on the device.  A label outside [0, C) contributes
 * neither loss nor gradient; it is reported as MPT_ERR_INVALID_ARG by the next
 * call that synchronises.  loss_host_or_null: if non-null the stream is
 * synchronised and the unscaled mean loss is stored.  MPT_ERR_STATE if no
 * mpt_forward preceded it. */
int mpt_backward_scaled(mpt_ctx *ctx, const int32_t *labels_dev, float *loss_host_or_null);

/* Master-weight pass (sections 3.1, 3.2).  With inv = 1.0f / S (one FP32 division on
 * the host): overflow = any element of any layer with non-finite f32(gW) * inv.
 * If overflow: nothing is modified.  Otherwise, per element, each operation rounded
 * separately in FP32 (no fused multiply-add):
 *   g = f32(gW) * inv ; [momentum: v = mu*v + g ; u = lr*v]  [plain: u = lr*g]
 *   w32 = w32 - u ; w16 = rn16(w32)
 * The skip decision is taken on the device.  overflow_host_or_null: if non-null
 * the stream is synchronised and 0/1 is stored.  Overflow is not an error: the
 * return value stays MPT_OK. */
int mpt_step(mpt_ctx *ctx, int *overflow_host_or_null);

/* Download one layer's FP32 master weights [out, in] (section 3.1).  Synchronous. */
int mpt_get_master(mpt_ctx *ctx, int layer, float *dst_host, size_t n);

/* One whole iteration from HOST buffers (figure 1 / section 3.1-3.2 in sequence):
 * copies x_host (FP16 [batch, in_1]) and labels_host (int32 [batch]) to the device
 * staging area, runs mpt_forward, mpt_backward_scaled and mpt_step, and returns
 * the loss and the overflow flag.  Synchronises the stream before returning. */
int mpt_train_step_host(mpt_ctx *ctx, const uint16_t *x_host, const int32_t *labels_host, int batch,
                        float *loss_host, int *overflow_host);

/* The same iteration with the host-to-device copy of a batch overlapped with the compute of
 * the previous one (the method's steps and arithmetic are those of mpt_train_step_host).
 * mpt_stage_batch_host copies x_host / labels_host into one of two staging slots on
 * copy_stream (a cudaStream_t of the caller, normally different from the context's stream) and
 * returns at once; host buffers must stay valid until that copy has run (use pinned memory for a
 * truly asynchronous copy).  mpt_train_step_staged makes the context's stream wait for the
 * oldest staged batch, runs forward, scaled backward and the master-weight pass on it,
 * synchronises and returns loss and overflow flag.  At most two batches can be staged;
 * staging a third, or stepping with none staged, returns MPT_ERR_STATE.  Typical loop:
 *   stage(batch 0); for t: stage(batch t+1); train_step_staged();                      */
int mpt_stage_batch_host(mpt_ctx *ctx, const uint16_t *x_host, const int32_t *labels_host, int batch,
                         void *copy_stream);
int mpt_train_step_staged(mpt_ctx *ctx, float *loss_host, int *overflow_host);

/* Change the loss scale (section 3.2) / learning rate; takes effect at the next
 * mpt_backward_scaled / mpt_step.  Same range checks as mpt_create. */
int mpt_set_scale(mpt_ctx *ctx, float S);
int mpt_set_lr(mpt_ctx *ctx, float lr);

/* Dynamic loss scaling (section 5 proposes adjusting S up or down from the overflow history of
 * the weight gradients, with overflowing steps skipped; it gives no schedule).  The schedule
 * taken here: after a
 * step that overflowed (and was skipped) S <- max(S/2, min_scale); after growth_interval
 * consecutive steps without overflow S <- min(2*S, max_scale); either event restarts the
 * count.  S stays a power of two if it starts as one, so scaling remains exact.  The scale
 * lives in device memory and is adjusted by a one-thread kernel at the end of mpt_step: no host
 * synchronisation is added.  enable = 0 returns to a constant scale (the current value).
 * mpt_get_scale synchronises and returns the scale the next backward pass will use. */
int mpt_set_dynamic_scale(mpt_ctx *ctx, int enable, int growth_interval, float min_scale, float max_scale);
int mpt_get_scale(mpt_ctx *ctx, float *S_out);

/* Test and checkpoint hooks.  mpt_get_tensor downloads an internal tensor without
 * padding (bytes must equal rows*cols*element size; ACT16/DACT16 use the batch of
 * the last forward; ACT16 layer l is a_{l+1}, the output of layer l).
 * mpt_set_grad overwrites one layer's FP16 weight gradient and refreshes the
 * device overflow flag over all layers.  mpt_set_momentum uploads an FP32
 * momentum buffer (checkpoint restore).  All synchronous. */
int mpt_get_tensor(mpt_ctx *ctx, int kind, int layer, void *dst_host, size_t bytes);
int mpt_set_grad(mpt_ctx *ctx, int layer, const uint16_t *src_host, size_t n);
int mpt_set_momentum(mpt_ctx *ctx, int layer, const float *src_host, size_t n);
/* Checkpoint hooks for Adam: the second state of a layer, and the running products beta1^t,
 * beta2^t (both 1 before the first applied step).  Synchronous. */
int mpt_set_state2(mpt_ctx *ctx, int layer, const float *src_host, size_t n);
int mpt_get_adam_products(mpt_ctx *ctx, float *b1t_out, float *b2t_out);
int mpt_set_adam_products(mpt_ctx *ctx, float b1t, float b2t);
/* Norm of the unscaled gradients and clipping coefficient of the last mpt_step (contexts created
 * with clip_norm > 0; MPT_ERR_STATE otherwise).  After an overflowing step the norm is inf or NaN
 * and the step was skipped.  Synchronous. */
int mpt_get_grad_norm(mpt_ctx *ctx, float *norm_out, float *coef_out);

/* Number of kernels this context has launched since creation (bookkeeping for
 * benchmarks). */
int mpt_launch_count(mpt_ctx *ctx, long long *count_out);

/* Per-kernel timing with CUDA events on the context's stream, for benchmarks.
 * mpt_profile(ctx, 1) synchronises, clears the counters and starts bracketing every
 * kernel launch of this context with a pair of events; mpt_profile(ctx, 0) stops.
 * mpt_profile_read synchronises and returns, per kernel class (MPT_PROF_*), the
 * summed device time in milliseconds, the summed algorithmic work (GEMM: 2*M*N*K
 * flop; update: 12 or 20 bytes per parameter; softmax: 4 bytes per logit) and the
 * number of launches since profiling was enabled.  Each array has
 * MPT_PROF_CLASSES entries. */
#define MPT_PROF_GEMM 0
#define MPT_PROF_UPDATE 1
#define MPT_PROF_SOFTMAX 2
#define MPT_PROF_OTHER 3
#define MPT_PROF_CLASSES 4
int mpt_profile(mpt_ctx *ctx, int enable);
int mpt_profile_read(mpt_ctx *ctx, double *ms_out, double *work_out, long long *launches_out);

/* Message for the last non-OK status of this context (never null). */
const char *mpt_last_error(mpt_ctx *ctx);

/* Releases the host-side context.  Does not touch device memory. */
void mpt_destroy(mpt_ctx *ctx);

/* ------------------------------------------------- stateless kernel launchers */

/* One FP16 product with FP32 accumulation and FP16 store (section 3.3).
 * op selects the stored layouts (see MPT_OP_*).  lda/ldb/ldc/ldmask are row
 * pitches in elements.  mask_dev (may be null): FP16 [M,N]; outputs where the
 * stored value is not > 0 are written as +0 (ReLU derivative from the stored
 * activation).  nonfinite_flag_dev (may be null): a uint32 that is OR-ed with 1 if
 * any stored output is inf or NaN (section 3.2: overflow shows up in the weight
 * gradients).  The tcgen05 kernel needs 16-byte aligned base pointers and pitches
 * that are multiples of 8 elements; other operands run on the CUDA-core kernel.
 * Results are run-to-run identical on a given GPU (no atomics in values; the order in which a
 * tile's k-blocks are accumulated is fixed by the tile's place in the kernel's work list).
 * status_dev: device uint32[4] scratch the kernel writes its error word into
 * (index 0: 0 = fine, else a timeout code); may be null to skip reporting. */
int mpt_gemm_f16(int op, int M, int N, int K, const uint16_t *A_dev, int lda, const uint16_t *B_dev,
                 int ldb, uint16_t *C_dev, int ldc, unsigned flags, const uint16_t *mask_dev,
                 int ldmask, uint32_t *nonfinite_flag_dev, uint32_t *status_dev, void *cuda_stream);

/* The same product with a caller-provided scratch buffer that allows the contraction to be
 * split (section 3.3 arithmetic unchanged except for the order of the FP32 additions: the
 * parts are added in ascending order by a second kernel, so results stay run-to-run
 * identical).  Large products use the scratch too: the tiles left over for a last, partly
 * filled round of the CTA-pair kernel are split along K so that the round takes a fraction of a
 * tile's time.  Outputs with few tiles and a long contraction (for instance 2048 x 1024 with
 * K = 8192) otherwise leave most SMs idle.  mpt_gemm_workspace_bytes returns the scratch size
 * the library would like for a shape (0 when it would not split); a smaller or null buffer
 * simply disables or narrows the split.  splitk_ws_dev must be 16-byte aligned. */
int mpt_gemm_workspace_bytes(int op, int M, int N, int K, size_t *bytes_out);
int mpt_gemm_f16_ws(int op, int M, int N, int K, const uint16_t *A_dev, int lda, const uint16_t *B_dev, int ldb,
                    uint16_t *C_dev, int ldc, unsigned flags, const uint16_t *mask_dev, int ldmask,
                    uint32_t *nonfinite_flag_dev, uint32_t *status_dev, void *splitk_ws_dev, size_t splitk_ws_bytes,
                    void *cuda_stream);

/* w16[e] = rn16(w32[e]) (section 3.1: the FP16 copy is made by rounding). */
int mpt_recast(const float *w32_dev, uint16_t *w16_dev, size_t n, void *cuda_stream);

/* Overflow inspection alone (section 3.2): *flag_dev |= 1 if any f32(g16[e]) * inv_S
 * is inf/NaN.  flag_dev must have been zeroed by the caller. */
int mpt_grad_nonfinite(const uint16_t *g16_dev, size_t n, float inv_S, uint32_t *flag_dev,
                       void *cuda_stream);

/* Master-weight pass over flat arrays (sections 3.1, 3.2), arithmetic as in mpt_step.
 * flags_dev: device uint32[2] scratch.  If detect != 0 the call first zeroes
 * flags_dev[0] and runs the inspection over g16 (an extra 2 bytes/element read);
 * if detect == 0 the caller has already produced flags_dev[0].  The update kernel
 * returns at once when flags_dev[0] != 0, otherwise updates in a single pass that
 * reads g16, w32, (v) once and writes w32, (v), w16 once, and stores its own
 * inspection result in flags_dev[1].  v_dev may be null iff use_momentum == 0. */
int mpt_update_flat(const uint16_t *g16_dev, float *w32_dev, float *v_dev, uint16_t *w16_dev, size_t n,
                    float inv_S, float lr, float mu, int use_momentum, int detect, uint32_t *flags_dev,
                    void *cuda_stream);

/* The same pass for any optimizer of mpt_optimizer (kind, weight decay, clipping).  s1_dev /
 * s2_dev: FP32 states (null when the kind does not use them).  b1t / b2t: for Adam, beta1^t and
 * beta2^t INCLUDING this step (the caller keeps the products); ignored otherwise.
 * clip_scratch_dev: needed iff opt->clip_norm > 0 (else may be null): MPT_CLIP_SCRATCH_BYTES of
 * device memory, 256-byte aligned, owned by the caller; the norm is taken over g16[0..n) and on
 * return (stream order) its first two floats hold the coefficient and the norm. */
#define MPT_CLIP_SCRATCH_BYTES 16384
int mpt_update_flat_opt(const mpt_optimizer *opt, const uint16_t *g16_dev, float *w32_dev, float *s1_dev, float *s2_dev,
                        uint16_t *w16_dev, size_t n, float inv_S, float b1t, float b2t, int detect, uint32_t *flags_dev,
                        void *clip_scratch_dev, void *cuda_stream);

/* ------------------------------------------------------------ LSTM layer with projection
 *
 * The recurrent layer of the paper's language model (section 4.5: 8192 cells projected to 1024)
 * in the mixed-precision recipe: FP16 storage, recurrent products with FP32 accumulation
 * (section 3.3), point-wise gate arithmetic in FP32 on the accumulators (section 3.3 leaves the
 * precision of memory-bound point-wise work open), reductions in FP32.  Per time step t:
 *   pre   = [x_t ; r_{t-1}] . Wg^T + bias         FP32 (never stored)
 *   i, f, o = sigmoid(pre_0, pre_1, pre_3), g = tanh(pre_2);  sigmoid(x) = 1/(1+exp(-x))
 *   c_t   = rn16(f*c_{t-1} + i*g)                 h_t = rn16(o * tanh(c_t as stored))
 *   r_t   = rn16(h_t . Wp^T)
 * Wg is [4H, I+P] with GATE-INTERLEAVED rows: row 4j+q is gate q of cell j (q: 0 input,
 * 1 forget, 2 candidate, 3 output); bias16, acts, dG and dWg use the same order.  The gate
 * arithmetic runs in the epilogue of the gate product: the pre-activations never reach memory.
 * Backward (scaled gradients, section 3.2), t = T-1 .. 0:
 *   drtot_t = rn16(dr_ext_t + recurrent part of dxr_{t+1})      dh_t = rn16(drtot_t . Wp)
 *   dc  = (dh*o)*(1 - tanh(c_t)^2) + dc_next ;  dG_t = rn16 of
 *         i: (dc*g)*(i*(1-i))  f: (dc*c_{t-1})*(f*(1-f))  g: (dc*i)*(1-g*g)  o: (dh*tanh(c_t))*(o*(1-o))
 *   dc_prev = rn16(dc*f) ;  dxr_t = rn16(dG_t . Wg)
 * and once, over all T*B rows (the sum over time is accumulated in FP32 inside one product):
 *   dWg = rn16(dG^T . xr)   dWp = rn16(drtot^T . h)   dbias = rn16(FP32 column sums of dG)
 * Every FP32 operation is rounded separately in the order written.
 *
 * All pointers are device memory owned by the caller; nothing is allocated.  Row-major, dense
 * (pitch = row length).  I, H and P must be multiples of 8 (MPT_ERR_SHAPE otherwise); the
 * tensor-core kernels are used when the product shapes allow, CUDA-core kernels otherwise. */
typedef struct mpt_lstm_desc {
    int32_t T, B;       /* time steps, rows per step (batch) */
    int32_t I, H, P;    /* input width, cells, projection width */
} mpt_lstm_desc;

typedef struct mpt_lstm_tensors {
    /* parameters (FP16 working copies) */
    const uint16_t *Wg16;    /* [4H, I+P] */
    const uint16_t *bias16;  /* [4H] */
    const uint16_t *Wp16;    /* [P, H] */
    /* forward: caller fills xr[t][:, :I] = x_t (t < T), xr[0][:, I:] = r_{-1}, c[0] = c_{-1};
     * the forward pass writes xr[t+1][:, I:] = r_t, c[t+1], h[t], acts[t] */
    uint16_t *xr;            /* [T+1, B, I+P] */
    uint16_t *c;             /* [T+1, B, H] */
    uint16_t *h;             /* [T, B, H] */
    uint16_t *acts;          /* [T, B, 4H] gate activations kept for the backward pass */
    /* backward */
    const uint16_t *dr_ext;  /* [T, B, P] scaled gradient wrt r_t from the consumer of the layer */
    uint16_t *dxr;           /* [T, B, I+P]: [:, :I] gradient wrt x_t, [:, I:] recurrent gradient wrt r_{t-1} */
    uint16_t *drtot;         /* [T, B, P] */
    uint16_t *dG;            /* [T, B, 4H] */
    uint16_t *dh;            /* [B, H] scratch */
    uint16_t *dc;            /* [2, B, H] scratch */
    uint16_t *dWg16;         /* [4H, I+P] */
    uint16_t *dWp16;         /* [P, H] */
    uint16_t *dbias16;       /* [4H] */
    float *bias_parts;       /* [8, 4H] FP32 scratch: bias-gradient partial sums in the backward pass; the forward
                              * pass keeps an FP32 copy of the bias in its first 4H entries (may be null there) */
    uint32_t *nonfinite_flag; /* one word, OR-ed with 1 when a weight or bias gradient is inf/NaN (section 3.2);
                                the caller zeroes it before mpt_lstm_backward */
    uint32_t *status_dev;    /* MPT status block of >= 16 words (first device-side error at word 3) or null */
    void *splitk_ws;         /* optional scratch that lets the projection product split its long contraction */
    size_t splitk_ws_bytes;  /* (mpt_gemm_workspace_bytes(MPT_OP_FWD, B, P, H) bytes; null / 0: never split) */
} mpt_lstm_tensors;

/* Forward over all T steps: 2T launches on the stream (gate product with fused gate epilogue,
 * projection product).  Reads Wg16, bias16, Wp16, xr, c[0]; writes h, acts, c[1..T], xr[1..T][:, I:]. */
int mpt_lstm_forward(const mpt_lstm_desc *desc, const mpt_lstm_tensors *t, void *cuda_stream);

/* Backward over all T steps, then the weight and bias gradients.  Needs the tensors the forward
 * pass wrote.  Writes dxr, drtot, dG, dWg16, dWp16, dbias16. */
int mpt_lstm_backward(const mpt_lstm_desc *desc, const mpt_lstm_tensors *t, void *cuda_stream);

/* The pieces on their own (same arithmetic).  mpt_lstm_cell_forward: one time step's gate product
 * with the fused gate epilogue; xr [B, K] pitch ldxr, Wg [4H, K] pitch ldw, acts [B, 4H] pitch
 * ldacts, c_prev/c_out/h_out [B, H] with their pitches.  mpt_lstm_cell_backward: dc_next may be
 * null (last step).  mpt_bias_grad: parts = FP32 scratch [8, cols].  mpt_add_f16: out = rn16(a+b). */
int mpt_lstm_cell_forward(int B, int H, int K, const uint16_t *xr, int ldxr, const uint16_t *Wg, int ldw,
                          const uint16_t *bias16, const uint16_t *c_prev, int ldcp, uint16_t *acts, int ldacts,
                          uint16_t *c_out, int ldco, uint16_t *h_out, int ldh, unsigned flags, uint32_t *status_dev,
                          void *cuda_stream);
int mpt_lstm_cell_backward(int B, int H, const uint16_t *dh, int lddh, const uint16_t *dc_next, int lddc,
                           const uint16_t *acts, int ldacts, const uint16_t *c_prev, int ldcp, const uint16_t *c16, int ldc,
                           uint16_t *dG, int lddg, uint16_t *dc_prev, int lddcp, void *cuda_stream);
int mpt_bias_grad(const uint16_t *dG, size_t rows, int cols, int ld, float *parts, uint16_t *db16,
                  uint32_t *nonfinite_flag, void *cuda_stream);
int mpt_add_f16(const uint16_t *a, int lda, const uint16_t *b, int ldb, uint16_t *out, int ldo, int rows, int cols,
                void *cuda_stream);

/* ------------------------------------------------------------ the LSTM layer, trained
 *
 * The layer above with everything section 3 asks of a trained layer: FP32 master copies of Wg,
 * Wp and the bias with FP16 working copies re-rounded after every applied step (section 3.1), a
 * loss multiplied by S before back-propagation, weight gradients unscaled and inspected for
 * inf/NaN with the step skipped on overflow (section 3.2; the paper's language model, section
 * 4.5, is its loss-scaling showcase: S = 128, Adagrad), optionally the dynamic scale schedule of
 * mpt_set_dynamic_scale.  One call runs one iteration on a batch of T*B rows:
 *   1. x_t into the step rows, r_{-1} = 0, c_{-1} = 0, then mpt_lstm_forward
 *   2. softmax cross-entropy over the projected outputs r_t taken as logits over P classes, one
 *      label per (t, b) row, mean over all T*B rows; dr_ext = rn16((p - onehot) * S / (T*B))
 *      (the arithmetic of mpt_softmax_ce)
 *   3. mpt_lstm_backward; the overflow word is OR-ed by the epilogues of dWg, dWp and dbias
 *   4. the optimizer step of mpt_update_flat_opt over the flat arena [Wg | Wp | bias] (one launch;
 *      every mpt_optimizer kind, weight decay, global-norm clipping), then the scale schedule
 * The workspace (mpt_lstm_workspace_bytes, 256-byte aligned, caller-owned) holds all parameters,
 * optimizer state, activations and gradients; nothing is allocated.  Asynchronous on the stream
 * unless loss_host / overflow_host is non-null (then the stream is synchronised and the unscaled
 * mean loss / the 0-1 skip flag of this iteration are written).  Error codes and the poisoned
 * state after MPT_ERR_CUDA / MPT_ERR_TIMEOUT are those of mpt_ctx; labels outside [0, P) contribute
 * nothing and are reported as MPT_ERR_INVALID_ARG by a synchronising call, after the step ran.
 * mpt_lstm_get_tensor kinds: masters (FP32), working copies, gradients of the last iteration
 * (FP16, scaled by S), first optimizer state (FP32), the step rows xr [T+1, B, I+P] whose right
 * columns hold r_t, and dr_ext [T, B, P]; the byte count must match exactly. */
typedef struct mpt_lstm_ctx mpt_lstm_ctx;
#define MPT_LSTM_T_WG32 0
#define MPT_LSTM_T_WP32 1
#define MPT_LSTM_T_BIAS32 2
#define MPT_LSTM_T_WG16 3
#define MPT_LSTM_T_WP16 4
#define MPT_LSTM_T_BIAS16 5
#define MPT_LSTM_T_DWG16 6
#define MPT_LSTM_T_DWP16 7
#define MPT_LSTM_T_DBIAS16 8
#define MPT_LSTM_T_S1_WG32 9
#define MPT_LSTM_T_S1_WP32 10
#define MPT_LSTM_T_S1_BIAS32 11
#define MPT_LSTM_T_XR16 12
#define MPT_LSTM_T_DREXT16 13
int mpt_lstm_workspace_bytes(const mpt_lstm_desc *desc, const mpt_optimizer *opt, size_t *bytes_out);
int mpt_lstm_create(const mpt_lstm_desc *desc, float S, const mpt_optimizer *opt, void *workspace_dev,
                    size_t workspace_bytes, void *cuda_stream, mpt_lstm_ctx **out);
/* Masters from HOST arrays Wg [4H, I+P] (gate-interleaved rows), bias [4H], Wp [P, H]; rounds the
 * working copies and zeroes the optimizer state.  Synchronous. */
int mpt_lstm_set_params(mpt_lstm_ctx *ctx, const float *Wg_host, const float *bias_host, const float *Wp_host);
/* x_dev: FP16 [T, B, I] dense; labels_dev: int32 [T*B], row t*B + b. */
int mpt_lstm_train_step(mpt_lstm_ctx *ctx, const uint16_t *x_dev, const int32_t *labels_dev, float *loss_host,
                        int *overflow_host);
int mpt_lstm_get_tensor(mpt_lstm_ctx *ctx, int kind, void *dst_host, size_t bytes);
int mpt_lstm_set_dynamic_scale(mpt_lstm_ctx *ctx, int enable, int growth_interval, float min_scale, float max_scale);
int mpt_lstm_get_scale(mpt_lstm_ctx *ctx, float *S_out);
const char *mpt_lstm_last_error(mpt_lstm_ctx *ctx);
void mpt_lstm_destroy(mpt_lstm_ctx *ctx);

/* Softmax cross-entropy forward and scaled backward (sections 3.2, 3.3), arithmetic
 * as in mpt_backward_scaled.  z_dev/dz_dev: FP16 [B, C] with pitches ldz/lddz
 * (the two must not overlap).  row_loss_dev: float [B] scratch; loss_dev: one float,
 * receives the unscaled mean; bad_labels_dev: one uint32, receives the number of
 * labels outside [0, C) (may be null).  status_dev (may be null): one uint32 the caller has
 * zeroed; the kernel that stages rows with asynchronous bulk copies writes a non-zero
 * time-out code there if one of its bounded waits runs out (rows are then left unwritten). */
int mpt_softmax_ce(const uint16_t *z_dev, int ldz, const int32_t *labels_dev, int B, int C, float S,
                   uint16_t *dz_dev, int lddz, float *row_loss_dev, float *loss_dev,
                   uint32_t *bad_labels_dev, uint32_t *status_dev, void *cuda_stream);

/* mpt_softmax_ce without the caller-provided scratch.  (The paper has no counterpart:
 * this entry point exists for the sake of callers, not of the method.)
 *
 * Some callers cannot obtain device memory at the point where they need the loss: code
 * that runs inside a framework which hands it a fixed set of tensors and owns every
 * other byte of the GPU, or a latency-critical loop that must not call cudaMalloc
 * because that call synchronises the whole device.  mpt_softmax_ce asks such a caller
 * for a float[B] scratch buffer it may not have.  This variant computes exactly the
 * same results (same kernels, same arithmetic) but keeps the per-row losses in a
 * fixed array inside the library, so the caller passes only inputs and outputs.
 * It calls no cudaMalloc/cudaFree and no allocating library routine.
 *
 *   - Limit: B <= MPT_SOFTMAX_STATIC_MAX_ROWS (65536 rows, a 256 KiB array that every
 *     GPU which loads the library holds until the process exits).  A larger B returns
 *     MPT_ERR_SHAPE and launches nothing; use mpt_softmax_ce for such batches.
 *   - The first call made on a device looks up the array's device address (a host-side
 *     runtime query, done once per device with that device current).  Make that first
 *     call during set-up, before any stream capture.  The stream must belong to the
 *     current device (the address looked up is the current device's): a stream of another
 *     device returns MPT_ERR_INVALID_ARG.
 *   - All calls on a GPU share the one array.  Two calls whose kernels overlap on the
 *     GPU (different streams, or different threads) race on it and may return wrong
 *     losses; calls on one stream are ordered and safe.  The array keeps the previous
 *     call's values, which is harmless: each call overwrites rows 0..B-1 before reading
 *     them and reads nothing else.
 * Other arguments, results and error codes are those of mpt_softmax_ce. */
#define MPT_SOFTMAX_STATIC_MAX_ROWS 65536
int mpt_softmax_ce_static(const uint16_t *z_dev, int ldz, const int32_t *labels_dev, int B, int C, float S,
                          uint16_t *dz_dev, int lddz, float *loss_dev, uint32_t *bad_labels_dev,
                          uint32_t *status_dev, void *cuda_stream);

/* Self-test of the bounded device-side waits (no counterpart in the paper: its only failure is
 * the gradient overflow of section 3.2).  Every pipeline kernel of this library waits on its
 * barriers for a limited time (2 s), then records a code in a status word and returns, so that
 * a fault in a copy or a peer can never hang the GPU.  These two calls make exactly that
 * happen on purpose, harmlessly: one CTA waits limit_us microseconds (1 .. 2,000,000) on a
 * barrier that nothing signals, gives up, writes its code and exits; the CUDA context stays
 * usable.
 *   mpt_selftest_wait_timeout      stateless.  status_dev: one uint32 the caller has zeroed.
 *                                  Synchronises the stream and returns MPT_ERR_TIMEOUT when the
 *                                  kernel reported the expiry (the expected outcome; the word is
 *                                  left set), MPT_OK if the word stayed zero.
 *   mpt_selftest_wait_timeout_ctx  the same through a context: the code lands in the context's
 *                                  status block, the call returns MPT_ERR_TIMEOUT and the context
 *                                  is poisoned exactly as after a real expiry (only
 *                                  mpt_last_error and mpt_destroy succeed afterwards). */
int mpt_selftest_wait_timeout(unsigned limit_us, uint32_t *status_dev, void *cuda_stream);
int mpt_selftest_wait_timeout_ctx(mpt_ctx *ctx, unsigned limit_us);

/* ------------------------------------------------------------ data-parallel step
 *
 * The paper's language model aggregates its batch over 4 GPUs (section 4.5); it gives no formulas
 * for the exchange.  Here R replicas hold identical FP16 weights, each runs forward and scaled
 * backward on its part of the batch, and ONE kernel per replica then does the gradient exchange,
 * the master-weight pass and the weight broadcast for that replica's shard of the parameters:
 *
 *   shard:   mpt_dp_shard(n, R, q) = elements [lo, hi) owned by replica q; per-replica length is
 *            ceil(ceil(n/8)/R)*8 (a multiple of 8, so every shard starts 16-byte aligned within
 *            16-byte aligned arrays), the last shards may be short or empty
 *   skip:    if ANY replica's overflow word is non-zero, nothing is written except flags_dev[0] = 1
 *            (section 3.2: the step is skipped everywhere); the per-replica words are what the
 *            weight-gradient epilogues (or mpt_grad_nonfinite) produced on each replica
 *   element e of the shard, each line one separately rounded FP32 operation:
 *            s = f32(g_0[e]) ; s = s + f32(g_q[e]) for q = 1 .. R-1 in ascending order
 *            g = s * inv_SR          inv_SR = 1 / (S * R): one FP32 multiplication, one division
 *            v = mu * v + g ; w32 = w32 - lr * v      (mu == 0 and v null: w32 = w32 - lr * g)
 *            h = rn16(w32) ; w16_q[e] = h for every replica q (its own copy included)
 *   The sum stays in FP32, so finite terms cannot overflow it.  Only the shard owner holds FP32
 *   state for its shard: w32_shard / v_shard point at element lo (a replica may allocate the shard
 *   alone, 8 instead of 8*R bytes per parameter across the job).
 *
 * g16_peers / flag_peers / w16_peers are HOST arrays of R DEVICE pointers in replica order; entry
 * `rank` is this replica's own buffer, the others are peer mappings of the other replicas' buffers
 * (all replicas use the same layout, n elements each).  Each gradient element crosses the link
 * once (read by its owner), each FP16 weight once per peer (written by its owner); the kernel
 * never waits on another replica.  Ordering is the caller's job: every replica's gradients and
 * overflow word must be complete before any replica calls this, and every replica's call must
 * have completed before any replica reads its weights or clears its overflow word (a stream-
 * ordered barrier across the replicas on both sides).  flags_dev: device uint32[2] of this
 * replica; [0] receives the OR of all replicas' words, [1] (zeroed by the call) the kernel's own
 * inspection of the unscaled mean gradients it formed.  flags_dev may be the same memory as
 * flag_peers[rank]: the kernel only ever sets bits there.
 * Errors: MPT_ERR_INVALID_ARG for R outside [1, MPT_DP_MAX_REPLICAS], rank outside [0, R), a null or
 * misaligned (16 bytes) pointer; MPT_ERR_CUDA if the launch fails. */
#define MPT_DP_MAX_REPLICAS 16
int mpt_dp_shard(size_t n, int R, int rank, size_t *lo_out, size_t *hi_out);
int mpt_dp_step_flat(const uint16_t *const *g16_peers, const uint32_t *const *flag_peers, uint16_t *const *w16_peers,
                     float *w32_shard_dev, float *v_shard_dev, size_t n, int R, int rank, float S, float lr, float mu,
                     uint32_t *flags_dev, void *cuda_stream);

/* The same step with any optimizer of mpt_optimizer on the mean gradient (weight decay, Nesterov,
 * Adagrad, Adam; op order as in mpt_update_flat_opt with g = s * inv_SR).  s1_shard / s2_shard:
 * the FP32 states of this replica's shard (null when the kind does not use them); b1t / b2t as in
 * mpt_update_flat_opt.
 * Global-norm clipping (section 3.2: after unscaling) bounds the norm of the MEAN gradient over all
 * n elements, which no single replica sees, so it takes two calls with the replicas ordered in
 * between: (1) every replica calls mpt_dp_norm_flat, which adds, in double over a fixed partition,
 * the squares of g = s * inv_SR over its own shard and stores the sum in *norm_slot_dev (a double in
 * memory the other replicas can map); scratch_dev: MPT_DP_NORM_SCRATCH_BYTES of this replica's own
 * memory, 8-byte aligned; (2) once every replica's call has completed, mpt_dp_step_flat_opt with
 * opt->clip_norm > 0 reads all R slots through norm_peers (HOST array of R DEVICE pointers, replica
 * order), adds them in ascending order, forms coef = min(1, clip_norm / (sqrt(total) + 1e-6)) rounded
 * to FP32 - the same bits on every replica - writes coef and the norm to clip_out_dev[0..1] (this
 * replica's memory) and multiplies every g by coef before weight decay and the step.  With
 * opt->clip_norm == 0 norm_peers and clip_out_dev are ignored (may be null). */
#define MPT_DP_NORM_SCRATCH_BYTES 8192
int mpt_dp_norm_flat(const uint16_t *const *g16_peers, size_t n, int R, int rank, float S, void *scratch_dev,
                     double *norm_slot_dev, void *cuda_stream);
int mpt_dp_step_flat_opt(const mpt_optimizer *opt, const uint16_t *const *g16_peers, const uint32_t *const *flag_peers,
                         uint16_t *const *w16_peers, float *w32_shard_dev, float *s1_shard_dev, float *s2_shard_dev, size_t n,
                         int R, int rank, float S, float b1t, float b2t, uint32_t *flags_dev,
                         const double *const *norm_peers, float *clip_out_dev, void *cuda_stream);

/* Data-parallel training of an mpt_ctx.  mpt_dp_layout_of reports where, inside the context's
 * workspace, the buffers live that the replicas exchange: byte offsets from the workspace base of
 * the scaled FP16 gradient arena, the FP16 weight arena and the overflow word (followed by the
 * word that receives the kernel's own inspection), and n, the arenas' length in elements.
 * Contexts created from the same description have the same layout, so a replica that has mapped a
 * peer's workspace forms that peer's pointers as mapped base + offset.
 * mpt_dp_attach: from now on mpt_step runs the kernel of mpt_dp_step_flat over the arenas instead
 * of the single-GPU master pass.  Entry `rank` of each array must be this context's own buffer.
 * The FP32 master weights and momentum are then current only inside this replica's shard
 * (mpt_get_master returns stale values outside it); the FP16 weights are complete on every
 * replica.  Every optimizer kind and weight decay are supported.  Global-norm clipping (contexts
 * created with clip_norm > 0) needs one more call and one more ordering point per iteration: after
 * mpt_backward_scaled every replica calls mpt_dp_norm (its shard of the squared norm of the mean
 * gradient, published in its status block next to the overflow word, so no further pointer table is
 * needed); when every replica's mpt_dp_norm has completed, mpt_step forms the common coefficient
 * from all replicas' values (mpt_step without that call: MPT_ERR_STATE); mpt_get_grad_norm then
 * returns the norm of the mean gradient.  Dynamic loss scaling works unchanged: every replica sees the same OR-ed
 * overflow word and moves its scale identically; the kernel reads S from device memory.  The
 * caller orders the replicas around mpt_step as described for mpt_dp_step_flat (before: every
 * replica's mpt_backward_scaled has completed; after: every replica's mpt_step has completed
 * before any replica's next mpt_forward).  R == 1 detaches (the arrays may then be null). */
typedef struct mpt_dp_layout {
    size_t g16_offset, w16_offset, flags_offset; /* bytes from the workspace base */
    size_t n;                                    /* elements in each arena */
} mpt_dp_layout;
int mpt_dp_layout_of(mpt_ctx *ctx, mpt_dp_layout *out);
int mpt_dp_attach(mpt_ctx *ctx, int R, int rank, const uint16_t *const *g16_peers, const uint32_t *const *flag_peers,
                  uint16_t *const *w16_peers);
int mpt_dp_norm(mpt_ctx *ctx);

/* A context that keeps FP32 state for its own shard only (sections 3.1 and 4.5: the master copy costs 4
 * bytes per parameter and every optimizer state another 4; with R replicas each needs them for 1/R of
 * the parameters, because a replica updates only its shard).  mpt_workspace_bytes_dp / mpt_create_dp are
 * mpt_workspace_bytes_opt / mpt_create_opt for replica `rank` of `replicas` (2 <= replicas <=
 * MPT_DP_MAX_REPLICAS): the FP32 master array and the optimizer-state arrays hold the elements
 * [lo, hi) of mpt_dp_shard(n, replicas, rank) of the flat parameter array (n from mpt_dp_layout_of) and
 * nothing else; all replicas' workspaces have the same size and layout.  Such a context
 *   - steps only while attached by mpt_dp_attach with the same replicas and rank (mpt_step otherwise:
 *     MPT_ERR_STATE; mpt_dp_attach with other values: MPT_ERR_INVALID_ARG);
 *   - mpt_set_master: rounds the whole layer into the FP16 weights (every replica must be given the
 *     same values) and keeps the FP32 values that fall inside the shard; it uses the gradient array as
 *     scratch, so gradients present are discarded;
 *   - mpt_set_momentum / mpt_set_state2 keep, and mpt_get_master / mpt_get_tensor(MASTER32, MOMENTUM32,
 *     STATE2_32) write, only the part of the layer inside the shard: elements [first, first + count) of
 *     the layer as mpt_state_range reports (count may be 0); the rest of the host buffer is not touched.
 *     Gathering a layer for a checkpoint is therefore one such call per replica into the same buffer.
 * mpt_state_range works on every context (first = 0, count = out*in for an ordinary one). */
int mpt_workspace_bytes_dp(const mpt_layer_desc *layers, int n_layers, int max_batch, const mpt_optimizer *opt, int replicas,
                           int rank, size_t *bytes_out);
int mpt_create_dp(const mpt_layer_desc *layers, int n_layers, float S, const mpt_optimizer *opt, int max_batch, int replicas,
                  int rank, void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out);
int mpt_state_range(mpt_ctx *ctx, int layer, size_t *first_out, size_t *count_out);

/* Exchange overlapped with the backward pass (section 4.5: the batch of one iteration is spread over several
 * GPUs; the gradient of a layer is final as soon as that layer's weight-gradient product has run, long
 * before the pass ends).  An attached context (mpt_dp_attach; one process per replica) can pull and add the
 * replicas' gradients layer by layer while the remaining layers are still being differentiated, and run
 * the master pass and the weight broadcast once the whole pass - and with it the overflow decision of
 * section 3.2 - is complete on every replica.  The arithmetic is that of mpt_dp_step_flat_opt (FP32 sum in
 * replica order, then the step), so the results are the same bits as without the overlap.
 *   mpt_dp_overlap_events: creates, once, one interprocess event per layer (and one more, see below) on this
 *     context and writes their handles ((n_layers + 1) x MPT_DP_HANDLE_BYTES, HOST) for the other replicas; mpt_backward_scaled then
 *     records event l on the context's stream after layer l's weight-gradient product.
 *   mpt_dp_overlap_attach: peer_handles = HOST array of R pointers to the other replicas' handle blocks
 *     (entry `rank` ignored); sum32_dev = DEVICE scratch of at least 4 bytes per element of this replica's
 *     shard (16-byte aligned, owned by the caller, must outlive the context's use of it).  Creates a second
 *     stream.  The handle blocks have n_layers + 1 entries: the last event marks the publication of this
 *     replica's part of the gradient norm (global-norm clipping).
 *   mpt_dp_reduce_async: enqueues, on the second stream, for each layer from the last to the first: waits
 *     on that layer's event of every replica, then the sum of the part of the layer inside this replica's
 *     shard.  Call it after mpt_backward_scaled has RETURNED on every replica (a host-side ordering point
 *     that need not wait for the GPUs: pass loss_host_or_null = NULL to mpt_backward_scaled so that it does
 *     not synchronise) - an event wait refers to the latest record enqueued before it.
 *     With global-norm clipping it also forms, from the sums, this replica's part of the squared norm of
 *     the mean gradient (as mpt_dp_norm does), publishes it and records the extra event; mpt_step must then be
 *     called after mpt_dp_reduce_async has RETURNED on every replica (one more host-side ordering point).
 *   mpt_step then waits (on the stream) for the sums and for every replica's last event (and norm event), and
 *     runs the step from the sums.  MPT_ERR_STATE if mpt_dp_reduce_async has not been called since the last step.
 * After mpt_step the replicas are ordered as for mpt_dp_attach.  Works with ordinary contexts and with
 * those of mpt_create_dp. */
int mpt_dp_overlap_events(mpt_ctx *ctx, uint8_t *handles_out);
int mpt_dp_overlap_attach(mpt_ctx *ctx, const uint8_t *const *peer_handles, float *sum32_dev, size_t sum32_bytes);
int mpt_dp_reduce_async(mpt_ctx *ctx);

/* Device memory that other processes can map (the buffers the replicas exchange).  mpt_dp_alloc
 * returns memory from the driver's allocator (not from a framework's pool, whose blocks cannot be
 * exported); mpt_dp_export writes an opaque MPT_DP_HANDLE_BYTES handle for the allocation that
 * contains dev_ptr - dev_ptr must be the pointer mpt_dp_alloc returned; mpt_dp_open maps another
 * PROCESS's allocation (on this or another GPU with peer access) and returns a device pointer
 * valid in the calling process; mpt_dp_close unmaps it.  The owner frees with mpt_dp_free only
 * after every peer has closed its mapping.  Errors: MPT_ERR_INVALID_ARG, MPT_ERR_CUDA. */
#define MPT_DP_HANDLE_BYTES 64
int mpt_dp_alloc(size_t bytes, void **dev_ptr_out);
int mpt_dp_free(void *dev_ptr);
int mpt_dp_export(const void *dev_ptr, uint8_t *handle_out);
int mpt_dp_open(const uint8_t *handle, void **dev_ptr_out);
int mpt_dp_close(void *dev_ptr);

/* Measurement aid (no counterpart in the paper): a one-warp kernel that measures the clock its SM
 * runs at, in MHz, by counting SM cycles over window_us (1 .. 100000) microseconds of the global
 * timer, and writes it to *mhz_dev (one float).  Asynchronous on the stream.  Enqueued before and
 * after a kernel it shows the clock that kernel ran at, which under a power cap changes from one
 * kernel of a training step to the next, far below the sampling period of nvidia-smi. */
int mpt_sm_clock_probe(unsigned window_us, float *mhz_dev, void *cuda_stream);

/* Library build identification, e.g. "mpt 0.1 sm_100a". */
const char *mpt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MPT_H_ */

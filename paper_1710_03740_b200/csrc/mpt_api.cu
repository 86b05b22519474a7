// C ABI of the library (include/mpt.h): host-side context, workspace carving,
// launch sequencing of one mixed-precision training iteration (paper sections
// 3.1-3.3), status handling.  No device memory is allocated here.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "mpt_common.cuh"

using namespace mpt;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layer {
    int in, out, relu;
    size_t off;      // element offset of this layer inside the flat parameter arenas
    size_t n;        // out * in
    int ld_out;      // row pitch (elements) of a_l / dz_l buffers
    uint16_t *act;   // a_{l+1}  [max_batch, ld_out]
    uint16_t *dact;  // dz_{l+1} [max_batch, ld_out]
};

struct Plan {
    size_t total = 0, P_pad = 0;
    size_t st_lo = 0, st_n = 0;      // elements [st_lo, st_lo + st_n) of the flat parameter array have FP32 state here
    size_t off_status = 0, off_master = 0, off_mom = 0, off_state2 = 0, off_w16 = 0, off_g16 = 0, off_x[2] = {0, 0},
           off_labels[2] = {0, 0}, off_rowloss = 0, off_norm = 0, off_splitk = 0, splitk_bytes = 0;
    std::vector<size_t> off_act, off_dact, lay_off;
    std::vector<int> ld_out;
};

int opt_states(const mpt_optimizer &o)
{
    switch (o.kind) {
        case MPT_OPT_SGD: return o.momentum != 0.0f ? 1 : 0;
        case MPT_OPT_NESTEROV:
        case MPT_OPT_ADAGRAD: return 1;
        default: return 2;
    }
}

bool valid_optimizer(const mpt_optimizer *o)
{
    if (!o) return false;
    if (o->kind < MPT_OPT_SGD || o->kind > MPT_OPT_ADAM) return false;
    if (!std::isfinite(o->lr)) return false;
    if (!(o->momentum >= 0.0f && o->momentum < 1.0f)) return false;
    if (!(o->weight_decay >= 0.0f) || !std::isfinite(o->weight_decay)) return false;
    if (!(o->clip_norm >= 0.0f) || !std::isfinite(o->clip_norm)) return false;
    if (o->kind == MPT_OPT_ADAM && !(o->beta2 >= 0.0f && o->beta2 < 1.0f)) return false;
    if ((o->kind == MPT_OPT_ADAM || o->kind == MPT_OPT_ADAGRAD) && (!(o->eps >= 0.0f) || !std::isfinite(o->eps))) return false;
    return true;
}

bool valid_scale(float S)
{
    return std::isfinite(S) && S >= 0x1p-100f && S <= 0x1p120f;
}

int validate_layers(const mpt_layer_desc *layers, int n_layers, int max_batch)
{
    if (!layers) return MPT_ERR_INVALID_ARG;
    if (n_layers < 1 || n_layers > 1024 || max_batch < 1) return MPT_ERR_SHAPE;
    for (int l = 0; l < n_layers; l++) {
        if (layers[l].in_features < 1 || layers[l].out_features < 1) return MPT_ERR_SHAPE;
        if (layers[l].relu != 0 && layers[l].relu != 1) return MPT_ERR_INVALID_ARG;
        if (l > 0 && layers[l].in_features != layers[l - 1].out_features) return MPT_ERR_SHAPE;
    }
    if (layers[n_layers - 1].relu != 0) return MPT_ERR_SHAPE;
    return MPT_OK;
}

void make_plan(const mpt_layer_desc *layers, int L, int max_batch, int n_states, Plan &pl, int replicas = 1, int rank = 0)
{
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    pl.off_status = take(ST_WORDS * sizeof(uint32_t));
    size_t P = 0;
    pl.lay_off.resize(L);
    for (int l = 0; l < L; l++) {
        pl.lay_off[l] = P;
        P += align_up((size_t)layers[l].in_features * layers[l].out_features, 128);
    }
    pl.P_pad = P;
    pl.st_lo = 0;
    pl.st_n = P;
    if (replicas > 1) {   // FP32 state of this replica's shard only
        size_t lo = 0, hi = 0;
        mpt_dp_shard(P, replicas, rank, &lo, &hi);
        pl.st_lo = lo;
        pl.st_n = hi - lo;
    }
    size_t state_elems = P;
    if (replicas > 1) {   // every replica reserves the size of the largest shard, so that all layouts are the same
        size_t lo0 = 0, hi0 = 0;
        mpt_dp_shard(P, replicas, 0, &lo0, &hi0);
        state_elems = hi0 - lo0;
    }
    const size_t state_bytes = (state_elems ? state_elems : 1) * 4;
    pl.off_master = take(state_bytes);
    pl.off_mom = n_states >= 1 ? take(state_bytes) : 0;
    pl.off_state2 = n_states >= 2 ? take(state_bytes) : 0;
    pl.off_w16 = take(P * 2);
    pl.off_g16 = take(P * 2);
    pl.off_act.resize(L); pl.off_dact.resize(L); pl.ld_out.resize(L);
    for (int l = 0; l < L; l++) {
        pl.ld_out[l] = (int)align_up((size_t)layers[l].out_features, 8);
        pl.off_act[l] = take((size_t)max_batch * pl.ld_out[l] * 2);
    }
    for (int l = 0; l < L; l++) pl.off_dact[l] = take((size_t)max_batch * pl.ld_out[l] * 2);
    for (int k = 0; k < 2; k++) {   // two staging slots: one being consumed, one being filled
        pl.off_x[k] = take((size_t)max_batch * layers[0].in_features * 2);
        pl.off_labels[k] = take((size_t)max_batch * 4);
    }
    pl.off_rowloss = take((size_t)max_batch * 4);
    pl.off_norm = take((size_t)kNormParts * sizeof(double));
    // scratch for split-K partial sums: the largest need of any product of the step that runs on
    // the single-CTA tensor-core kernel (small or thin outputs), capped at 256 MB
    size_t need_max = 0;
    for (int l = 0; l < L; l++) {
        const int B = max_batch, in = layers[l].in_features, out = layers[l].out_features;
        const int shapes[3][3] = {{B, out, in}, {out, in, B}, {B, in, out}};   // forward, wgrad, dgrad as (M, N, K)
        for (int k = 0; k < 3; k++) {
            if (k == 2 && l == 0) continue;
            size_t need = 0;
            tc_choose_pair(shapes[k][0], shapes[k][1], shapes[k][2], (size_t)256 << 20, &need);
            if (need > need_max) need_max = need;
        }
    }
    pl.splitk_bytes = need_max;
    pl.off_splitk = need_max ? take(need_max) : 0;
    pl.total = off;
}

}  // namespace

struct mpt_ctx {
    std::vector<Layer> layers;
    float S, lr, mu;
    bool use_momentum;          // first optimizer state in use
    int opt_kind = MPT_OPT_SGD;
    float beta2 = 0.0f, eps = 0.0f, wd = 0.0f, clip = 0.0f;
    float *state2 = nullptr;
    int max_batch;
    cudaStream_t stream;
    uint8_t *ws;
    Plan plan;
    uint32_t *status;
    float *master, *mom;
    uint16_t *w16, *g16, *x_stage[2];
    int32_t *labels_stage[2];
    float *splitk_ws = nullptr;
    // staged (pipelined) host batches: slot state and the events that order copies against compute
    cudaEvent_t staged_ev[2] = {nullptr, nullptr}, used_ev[2] = {nullptr, nullptr};
    bool staged_valid[2] = {false, false}, used_recorded[2] = {false, false};
    int staged_batch[2] = {0, 0};
    int stage_w = 0, stage_r = 0;
    float *row_loss;
    double *norm_parts;   // fixed-partition partial sums of the gradient norm (clipping)
    const uint16_t *x_cur = nullptr;
    int batch = 0;
    bool forward_done = false, have_grads = false, poisoned = false;
    long long launches = 0;
    bool disable_tc = false, disable_pair = false;
    // dynamic loss scaling (off by default: constant S)
    bool dynamic_scale = false;
    int growth_interval = 2000;
    float scale_backoff = 0.5f, scale_growth = 2.0f, scale_min = 0x1p-100f, scale_max = 0x1p120f;
    // data-parallel step (mpt_dp_attach): replica count (0 or 1: off), this replica, peer tables
    int dp_R = 0, dp_rank = 0;
    // mpt_create_dp: FP32 master and optimizer state exist for this replica's shard only; master / mom /
    // state2 are then bases such that element i of the flat array is at [i] for i inside the shard
    int shard_R = 0, shard_rank = 0;
    // overlapped exchange (mpt_dp_overlap_attach): the pull-and-sum of each layer's gradients runs on dp_stream
    // as soon as that layer's weight gradient is complete on every replica (interprocess events)
    bool dp_overlap = false, dp_reduced = false;
    cudaStream_t dp_stream = nullptr;
    std::vector<cudaEvent_t> ev_own;                      // per layer: this replica's weight gradient is complete
    std::vector<cudaEvent_t> ev_peer[MPT_DP_MAX_REPLICAS]; // the same events of the other replicas, opened here
    cudaEvent_t ev_reduced = nullptr;
    float *sum32 = nullptr;                               // FP32 sums over the replicas, this replica's shard
    bool dp_norm_done = false;   // mpt_dp_norm has run since the last backward pass (clipping in data-parallel mode)
    const uint16_t *dp_g16[MPT_DP_MAX_REPLICAS] = {};
    const uint32_t *dp_flag[MPT_DP_MAX_REPLICAS] = {};
    uint16_t *dp_w16[MPT_DP_MAX_REPLICAS] = {};
    std::string err;
    // optional per-kernel timing with CUDA events (mpt_profile)
    bool profiling = false;
    struct Span { cudaEvent_t a, b; int cls; };
    std::vector<Span> spans;
    std::vector<Span> pool;
    double prof_ms[MPT_PROF_CLASSES] = {0, 0, 0, 0};
    double prof_work[MPT_PROF_CLASSES] = {0, 0, 0, 0};
    long long prof_launches[MPT_PROF_CLASSES] = {0, 0, 0, 0};
};

namespace {

int fail(mpt_ctx *c, int code, const char *fmt, const char *detail = "")
{
    char buf[512];
    snprintf(buf, sizeof buf, fmt, detail);
    c->err = buf;
    if (code == MPT_ERR_CUDA || code == MPT_ERR_TIMEOUT) c->poisoned = true;
    return code;
}

int cuda_fail(mpt_ctx *c, cudaError_t e, const char *what)
{
    char buf[512];
    snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
    c->err = buf;
    c->poisoned = true;
    return MPT_ERR_CUDA;
}

#define CK(call, what)                                            \
    do {                                                          \
        cudaError_t e__ = (call);                                 \
        if (e__ != cudaSuccess) return cuda_fail(c, e__, what);   \
    } while (0)

int usable(mpt_ctx *c)
{
    if (!c) return MPT_ERR_INVALID_ARG;
    if (c->poisoned) return MPT_ERR_STATE;
    return MPT_OK;
}

// The loss scale lives in the status block (S, 1/S, clean-step counter): kernels read it from
// there, so it can change on the device (dynamic scaling) without a host round trip.
int push_scale(mpt_ctx *c)
{
    uint32_t w[3];
    const float inv = 1.0f / c->S;
    memcpy(&w[0], &c->S, 4);
    memcpy(&w[1], &inv, 4);
    w[2] = 0;
    CK(cudaMemcpyAsync(c->status + ST_SCALE, w, sizeof w, cudaMemcpyHostToDevice, c->stream), "scale upload");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int push_adam_products(mpt_ctx *c, float b1t, float b2t)
{
    uint32_t w[2];
    memcpy(&w[0], &b1t, 4);
    memcpy(&w[1], &b2t, 4);
    CK(cudaMemcpyAsync(c->status + ST_B1T, w, sizeof w, cudaMemcpyHostToDevice, c->stream), "optimizer state upload");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

// Brackets one kernel launch with CUDA events on the context's stream when profiling.
struct ProfSpan {
    mpt_ctx *c;
    bool on;
    mpt_ctx::Span sp;
    ProfSpan(mpt_ctx *ctx, int cls, double work) : c(ctx), on(ctx->profiling)
    {
        if (!on) return;
        if (!c->pool.empty()) { sp = c->pool.back(); c->pool.pop_back(); }
        else if (cudaEventCreate(&sp.a) != cudaSuccess || cudaEventCreate(&sp.b) != cudaSuccess) { on = false; return; }
        sp.cls = cls;
        c->prof_work[cls] += work;
        c->prof_launches[cls] += 1;
        cudaEventRecord(sp.a, c->stream);
    }
    ~ProfSpan()
    {
        if (!on) return;
        cudaEventRecord(sp.b, c->stream);
        c->spans.push_back(sp);
    }
};

// One product of the iteration, on the tensor-core kernel when the operands allow it.
int gemm(mpt_ctx *c, int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb, uint16_t *C,
         int ldc, bool relu, const uint16_t *mask, int ldmask, uint32_t *nonfinite)
{
    cudaError_t e;
    ProfSpan span(c, MPT_PROF_GEMM, 2.0 * M * N * K);
    if (!c->disable_tc && tc_gemm_supported(op, M, N, K, A, lda, B, ldb, C, ldc, mask, ldmask)) {
        const int split = c->disable_pair ? 0 : tc4_split_for(M, N, K);
        if (split)
            e = launch_gemm_tc4(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite, c->status + ST_KERNEL_ERR,
                                c->stream, split);
        else if (!c->disable_pair && tc_choose_pair(M, N, K, c->plan.splitk_bytes, nullptr))
            e = launch_gemm_tc2(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite,
                                c->status + ST_KERNEL_ERR, c->stream, nullptr, c->splitk_ws, c->plan.splitk_bytes);
        else
            e = launch_gemm_tc(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite,
                               c->status + ST_KERNEL_ERR, c->stream, c->splitk_ws, c->plan.splitk_bytes);
        c->launches += g_last_gemm_launches;
    } else {
        e = launch_gemm_simt(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite, c->stream);
        c->launches++;
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "gemm launch");
    return MPT_OK;
}

// After a stream synchronisation: read the status block once and turn device-side
// conditions into return codes.
int read_status(mpt_ctx *c, uint32_t (&st)[ST_WORDS])
{
    CK(cudaMemcpyAsync(st, c->status, sizeof st, cudaMemcpyDeviceToHost, c->stream), "status copy");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    if (st[ST_KERNEL_ERR] != 0) {
        char buf[64];
        snprintf(buf, sizeof buf, "0x%x", st[ST_KERNEL_ERR]);
        return fail(c, MPT_ERR_TIMEOUT, "a device-side bounded wait expired (code|cta<<8 = %s)", buf);
    }
    return MPT_OK;
}

int do_forward(mpt_ctx *c, const uint16_t *x_dev, int batch)
{
    if (batch < 1 || batch > c->max_batch) return fail(c, MPT_ERR_SHAPE, "batch outside [1, max_batch]");
    const uint16_t *a = x_dev;
    int lda = c->layers[0].in;
    for (size_t l = 0; l < c->layers.size(); l++) {
        Layer &ly = c->layers[l];
        int r = gemm(c, MPT_OP_FWD, batch, ly.out, ly.in, a, lda, c->w16 + ly.off, ly.in, ly.act, ly.ld_out, ly.relu != 0,
                     nullptr, 0, nullptr);
        if (r != MPT_OK) return r;
        a = ly.act;
        lda = ly.ld_out;
    }
    c->x_cur = x_dev;
    c->batch = batch;
    c->forward_done = true;
    return MPT_OK;
}

int do_backward(mpt_ctx *c, const int32_t *labels_dev)
{
    if (!c->forward_done) return fail(c, MPT_ERR_STATE, "mpt_backward_scaled needs a preceding mpt_forward");
    const int L = (int)c->layers.size(), B = c->batch;
    // status words 0..2 (overflow, overflow seen, bad labels) start the backward at zero
    CK(cudaMemsetAsync(c->status, 0, 3 * sizeof(uint32_t), c->stream), "status clear");
    Layer &last = c->layers[L - 1];
    int nl = 0;
    cudaError_t e;
    {
        ProfSpan span(c, MPT_PROF_SOFTMAX, 4.0 * B * last.out);
        e = launch_softmax_ce(last.act, last.ld_out, labels_dev, B, last.out, c->S, last.dact, last.ld_out, c->row_loss,
                              (float *)(c->status + ST_LOSS), c->status + ST_BAD_LABELS, c->stream, &nl,
                              (const float *)(c->status + ST_SCALE), c->status + ST_KERNEL_ERR);
    }
    c->launches += nl;
    if (e != cudaSuccess) return cuda_fail(c, e, "softmax launch");
    for (int l = L - 1; l >= 0; l--) {
        Layer &ly = c->layers[l];
        const uint16_t *a_prev = l ? c->layers[l - 1].act : c->x_cur;
        const int ld_prev = l ? c->layers[l - 1].ld_out : ly.in;
        int r = gemm(c, MPT_OP_WGRAD, ly.out, ly.in, B, ly.dact, ly.ld_out, a_prev, ld_prev, c->g16 + ly.off, ly.in, false,
                     nullptr, 0, c->status + ST_OVERFLOW);
        if (r != MPT_OK) return r;
        if (c->dp_overlap) CK(cudaEventRecord(c->ev_own[l], c->stream), "event record");
        if (l > 0) {
            Layer &pv = c->layers[l - 1];
            r = gemm(c, MPT_OP_DGRAD, B, ly.in, ly.out, ly.dact, ly.ld_out, c->w16 + ly.off, ly.in, pv.dact, pv.ld_out, false,
                     pv.relu ? pv.act : nullptr, pv.ld_out, nullptr);
            if (r != MPT_OK) return r;
        }
    }
    c->forward_done = false;
    c->have_grads = true;
    return MPT_OK;
}

int do_step(mpt_ctx *c)
{
    if (!c->have_grads) return fail(c, MPT_ERR_STATE, "mpt_step needs gradients (mpt_backward_scaled or mpt_set_grad)");
    if (c->shard_R > 1 && (c->dp_R != c->shard_R || c->dp_rank != c->shard_rank))
        return fail(c, MPT_ERR_STATE, "a context created by mpt_create_dp steps only while attached (mpt_dp_attach) as that replica");
    const float inv = 1.0f / c->S;
    CK(cudaMemsetAsync(c->status + ST_OVERFLOW_SEEN, 0, sizeof(uint32_t), c->stream), "status clear");
    cudaError_t e;
    if (c->dp_R > 1) {
        size_t lo = 0, hi = 0;
        mpt_dp_shard(c->plan.P_pad, c->dp_R, c->dp_rank, &lo, &hi);
        int nl = 0;
        const float *sums = nullptr;
        if (c->dp_overlap) {
            // the sums were formed on dp_stream (mpt_dp_reduce_async); the new weights may be written into a
            // replica only when its whole backward pass is complete (its last event)
            if (!c->dp_reduced) return fail(c, MPT_ERR_STATE, "overlapped exchange: call mpt_dp_reduce_async before mpt_step");
            CK(cudaStreamWaitEvent(c->stream, c->ev_reduced, 0), "event wait");
            for (int q = 0; q < c->dp_R; q++)
                if (q != c->dp_rank) CK(cudaStreamWaitEvent(c->stream, c->ev_peer[q][0], 0), "event wait");
            if (c->clip > 0.0f)      // every replica's part of the norm is published
                for (int q = 0; q < c->dp_R; q++)
                    if (q != c->dp_rank) CK(cudaStreamWaitEvent(c->stream, c->ev_peer[q][c->layers.size()], 0), "event wait");
            c->dp_reduced = false;
            sums = c->sum32;
        }
        if (c->clip > 0.0f) {
            // every replica adds all replicas' published shard sums in replica order: same coefficient everywhere
            if (!c->dp_norm_done)
                return fail(c, MPT_ERR_STATE, "clipping in data-parallel mode: call mpt_dp_norm on every replica (then order the replicas) before mpt_step");
            const double *slots[MPT_DP_MAX_REPLICAS];
            for (int q = 0; q < c->dp_R; q++) slots[q] = (const double *)(c->dp_flag[q] + (ST_DP_NORM - ST_OVERFLOW));
            e = launch_dp_clip_coef(slots, c->dp_R, c->clip, (float *)(c->status + ST_CLIP_COEF), c->stream);
            c->launches++;
            if (e != cudaSuccess) return cuda_fail(c, e, "clip launch");
            c->dp_norm_done = false;
        }
        {
            // bytes through this GPU's memory system: R gradients read, the shard's state, R weight copies written
            const double per_elem = 2.0 * c->dp_R + 8.0 + (c->use_momentum ? 8.0 : 0.0) + (c->state2 ? 8.0 : 0.0) + 2.0 * c->dp_R;
            ProfSpan span(c, MPT_PROF_UPDATE, per_elem * (double)(hi - lo));
            const float inv_SR = 1.0f / (c->S * (float)c->dp_R);
            const float *S_dev = (const float *)(c->status + ST_SCALE);
            if (!sums && c->opt_kind == MPT_OPT_SGD && c->wd == 0.0f && c->clip <= 0.0f)
                e = launch_dp_step(c->dp_g16, c->dp_flag, c->dp_w16, c->dp_R, c->master + lo, c->use_momentum ? c->mom + lo : nullptr,
                                   lo, hi - lo, inv_SR, S_dev, c->lr, c->use_momentum ? c->mu : 0.0f, c->status + ST_OVERFLOW,
                                   c->stream, &nl);
            else
                e = launch_dp_step_opt(c->opt_kind, c->dp_g16, c->dp_flag, c->dp_w16, c->dp_R, c->master + lo,
                                       c->mom ? c->mom + lo : nullptr, c->state2 ? c->state2 + lo : nullptr, lo, hi - lo, inv_SR,
                                       S_dev, c->lr, c->mu, c->beta2, c->eps, c->wd, 1.0f, 1.0f,
                                       c->opt_kind == MPT_OPT_ADAM ? (const float *)(c->status + ST_B1T) : nullptr,
                                       c->status + ST_OVERFLOW, c->stream, &nl,
                                       c->clip > 0.0f ? (const float *)(c->status + ST_CLIP_COEF) : nullptr, sums);
        }
        c->launches += nl;
        if (e != cudaSuccess) return cuda_fail(c, e, "data-parallel step launch");
    } else {
        const double bytes_per_param = 12.0 + 8.0 * (c->use_momentum ? 1 : 0) + 8.0 * (c->state2 ? 1 : 0) + (c->clip > 0.0f ? 2.0 : 0.0);
        ProfSpan span(c, MPT_PROF_UPDATE, bytes_per_param * (double)c->plan.P_pad);
        if (c->clip > 0.0f) {
            // norm over the whole gradient arena (layer padding holds zeros) and the coefficient
            e = launch_clip_coef(c->g16, c->plan.P_pad, inv, (const float *)(c->status + ST_INV_SCALE), c->clip, c->norm_parts,
                                 (float *)(c->status + ST_CLIP_COEF), c->stream);
            c->launches += 2;
            if (e != cudaSuccess) return cuda_fail(c, e, "clip launch");
        }
        if (c->opt_kind == MPT_OPT_SGD && c->wd == 0.0f && c->clip <= 0.0f)
            e = launch_update(c->g16, c->master, c->mom, c->w16, c->plan.P_pad, inv, c->lr, c->mu, c->use_momentum,
                              c->status + ST_OVERFLOW, c->stream, (const float *)(c->status + ST_INV_SCALE));
        else
            e = launch_update_opt(c->opt_kind, c->g16, c->master, c->mom, c->state2, c->w16, c->plan.P_pad, inv, c->lr, c->mu,
                                  c->beta2, c->eps, c->wd, 1.0f, 1.0f, c->status + ST_OVERFLOW, c->stream,
                                  (const float *)(c->status + ST_INV_SCALE),
                                  c->opt_kind == MPT_OPT_ADAM ? (const float *)(c->status + ST_B1T) : nullptr,
                                  c->clip > 0.0f ? (const float *)(c->status + ST_CLIP_COEF) : nullptr);
        c->launches++;
        if (e != cudaSuccess) return cuda_fail(c, e, "update launch");
    }
    if (c->dynamic_scale || c->opt_kind == MPT_OPT_ADAM) {
        // end-of-step bookkeeping on the device: loss scale and Adam's beta^t move only on applied steps
        ProfSpan span(c, MPT_PROF_OTHER, 0.0);
        e = launch_post_step(c->status, c->dynamic_scale ? c->growth_interval : 0, c->scale_backoff, c->scale_growth,
                             c->scale_min, c->scale_max, c->opt_kind == MPT_OPT_ADAM ? 1 : 0, c->mu, c->beta2, c->stream);
        c->launches++;
        if (e != cudaSuccess) return cuda_fail(c, e, "post-step launch");
    }
    return MPT_OK;
}

int finish_step(mpt_ctx *c, const uint32_t (&st)[ST_WORDS], int *overflow_host)
{
    if (st[ST_OVERFLOW] == 0 && st[ST_OVERFLOW_SEEN] != 0)
        return fail(c, MPT_ERR_INTERNAL, "update kernel saw a non-finite gradient the producer did not flag");
    if (overflow_host) *overflow_host = st[ST_OVERFLOW] ? 1 : 0;
    return MPT_OK;
}

}  // namespace

namespace mpt {

// Shape checks and kernel choice shared by the stateless product entry points and the LSTM layer:
// CTA-pair kernel for large outputs, single-CTA kernel (with optional split-K scratch) for the
// rest of what the tensor-core path takes, CUDA-core kernel otherwise.  lstm != null: forward
// product with the fused gate epilogue (tensor-core kernels only; the caller checks that first).
int dispatch_gemm(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb, uint16_t *C, int ldc,
                  unsigned flags, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag, uint32_t *status_dev,
                  void *splitk_ws_dev, size_t splitk_ws_bytes, cudaStream_t st, const LstmEpi *lstm)
{
    if (!A || !B || !C) return MPT_ERR_INVALID_ARG;
    if (op != MPT_OP_FWD && op != MPT_OP_DGRAD && op != MPT_OP_WGRAD) return MPT_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || K < 0) return MPT_ERR_SHAPE;
    if (M == 0 || N == 0) return MPT_OK;
    const int a_cols = op == MPT_OP_WGRAD ? M : K, b_cols = op == MPT_OP_FWD ? K : N;
    if (lda < a_cols || ldb < b_cols || ldc < N || (mask && ldmask < N)) return MPT_ERR_SHAPE;
    const bool relu = (flags & MPT_GEMM_RELU) != 0;
    bool tc_ok = K > 0 && tc_gemm_supported(op, M, N, K, A, lda, B, ldb, C, ldc, mask, ldmask);
    constexpr unsigned kForceSplit = MPT_GEMM_FORCE_SPLIT2 | MPT_GEMM_FORCE_SPLIT4;
    if (((flags & (MPT_GEMM_FORCE_TC | MPT_GEMM_FORCE_PAIR | MPT_GEMM_FORCE_PAIR512 | kForceSplit)) || lstm) && !tc_ok)
        return MPT_ERR_SHAPE;
    if ((flags & kForceSplit) && (lstm || K < ((flags & MPT_GEMM_FORCE_SPLIT4) ? 256 : 128))) return MPT_ERR_SHAPE;
    const unsigned forced = flags & (MPT_GEMM_FORCE_SIMT | MPT_GEMM_FORCE_TC | MPT_GEMM_FORCE_PAIR | MPT_GEMM_FORCE_PAIR512 | kForceSplit);
    const int auto_split = (tc_ok && !lstm && !forced) ? tc4_split_for(M, N, K) : 0;
    cudaError_t e;
    if (tc_ok && ((flags & kForceSplit) || auto_split)) {
        const int split = (flags & MPT_GEMM_FORCE_SPLIT4) ? 4 : ((flags & MPT_GEMM_FORCE_SPLIT2) ? 2 : auto_split);
        e = launch_gemm_tc4(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag, status_dev, st, split);
    } else if (tc_ok && !lstm && (flags & MPT_GEMM_FORCE_PAIR512)) {
        e = launch_gemm_tc3(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag, status_dev, st);
    } else if (tc_ok && !(flags & MPT_GEMM_FORCE_SIMT)) {
        const size_t ws_ok = (splitk_ws_dev && (((uintptr_t)splitk_ws_dev) & 15) == 0) ? splitk_ws_bytes : 0;
        const bool pair = (flags & MPT_GEMM_FORCE_PAIR) ||
                          (!(flags & MPT_GEMM_FORCE_TC) && (lstm ? tc2_gemm_preferred(M, N, K) : tc_choose_pair(M, N, K, ws_ok, nullptr)));
        if (pair)
            e = launch_gemm_tc2(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag, status_dev, st, lstm,
                                splitk_ws_dev, splitk_ws_bytes);
        else
            e = launch_gemm_tc(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag, status_dev, st,
                               (float *)splitk_ws_dev, splitk_ws_bytes, lstm);
    } else
        e = launch_gemm_simt(op, M, N, K, A, lda, B, ldb, C, ldc, relu, mask, ldmask, nonfinite_flag, st);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

// Part of a layer's parameters whose FP32 state this context holds: all of it, or, for a context made
// by mpt_create_dp, the part inside the replica's shard.  first is relative to the layer.
void state_part(const mpt_ctx *c, const Layer &ly, size_t *first, size_t *count)
{
    const size_t a = ly.off > c->plan.st_lo ? ly.off : c->plan.st_lo;
    const size_t e1 = ly.off + ly.n, e2 = c->plan.st_lo + c->plan.st_n;
    const size_t b = e1 < e2 ? e1 : e2;
    *first = a < b ? a - ly.off : 0;
    *count = a < b ? b - a : 0;
}

}  // namespace mpt

extern "C" {

const char *mpt_version(void) { return "mpt 0.1 sm_100a"; }

int mpt_workspace_bytes(const mpt_layer_desc *layers, int n_layers, int max_batch, int use_momentum, size_t *bytes_out)
{
    if (!bytes_out) return MPT_ERR_INVALID_ARG;
    int r = validate_layers(layers, n_layers, max_batch);
    if (r != MPT_OK) return r;
    Plan pl;
    make_plan(layers, n_layers, max_batch, use_momentum != 0 ? 1 : 0, pl);
    *bytes_out = pl.total;
    return MPT_OK;
}

int mpt_workspace_bytes_opt(const mpt_layer_desc *layers, int n_layers, int max_batch, const mpt_optimizer *opt,
                            size_t *bytes_out)
{
    if (!bytes_out || !opt) return MPT_ERR_INVALID_ARG;
    int r = validate_layers(layers, n_layers, max_batch);
    if (r != MPT_OK) return r;
    if (!valid_optimizer(opt)) return MPT_ERR_INVALID_ARG;
    Plan pl;
    make_plan(layers, n_layers, max_batch, opt_states(*opt), pl);
    *bytes_out = pl.total;
    return MPT_OK;
}

int mpt_create(const mpt_layer_desc *layers, int n_layers, float S, float lr, float momentum, int max_batch,
               void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out)
{
    mpt_optimizer opt = {MPT_OPT_SGD, lr, momentum, 0.0f, 0.0f, 0.0f, 0.0f};
    return mpt_create_opt(layers, n_layers, S, &opt, max_batch, workspace_dev, workspace_bytes, cuda_stream, out);
}

static int create_impl(const mpt_layer_desc *layers, int n_layers, float S, const mpt_optimizer *opt, int max_batch,
                       int replicas, int rank, void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out);

int mpt_create_opt(const mpt_layer_desc *layers, int n_layers, float S, const mpt_optimizer *opt, int max_batch,
                   void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out)
{
    return create_impl(layers, n_layers, S, opt, max_batch, 1, 0, workspace_dev, workspace_bytes, cuda_stream, out);
}

int mpt_workspace_bytes_dp(const mpt_layer_desc *layers, int n_layers, int max_batch, const mpt_optimizer *opt, int replicas,
                           int rank, size_t *bytes_out)
{
    if (!bytes_out || !opt) return MPT_ERR_INVALID_ARG;
    int r = validate_layers(layers, n_layers, max_batch);
    if (r != MPT_OK) return r;
    if (!valid_optimizer(opt)) return MPT_ERR_INVALID_ARG;
    if (replicas < 2 || replicas > MPT_DP_MAX_REPLICAS || rank < 0 || rank >= replicas) return MPT_ERR_INVALID_ARG;
    Plan pl;
    make_plan(layers, n_layers, max_batch, opt_states(*opt), pl, replicas, rank);
    *bytes_out = pl.total;
    return MPT_OK;
}

int mpt_create_dp(const mpt_layer_desc *layers, int n_layers, float S, const mpt_optimizer *opt, int max_batch, int replicas,
                  int rank, void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out)
{
    if (replicas < 2 || replicas > MPT_DP_MAX_REPLICAS || rank < 0 || rank >= replicas) {
        if (out) *out = nullptr;
        return MPT_ERR_INVALID_ARG;
    }
    return create_impl(layers, n_layers, S, opt, max_batch, replicas, rank, workspace_dev, workspace_bytes, cuda_stream, out);
}

static int create_impl(const mpt_layer_desc *layers, int n_layers, float S, const mpt_optimizer *opt, int max_batch,
                       int replicas, int rank, void *workspace_dev, size_t workspace_bytes, void *cuda_stream, mpt_ctx **out)
{
    if (!out) return MPT_ERR_INVALID_ARG;
    *out = nullptr;
    if (!workspace_dev) return MPT_ERR_INVALID_ARG;
    int r = validate_layers(layers, n_layers, max_batch);
    if (r != MPT_OK) return r;
    if (!valid_scale(S) || !valid_optimizer(opt)) return MPT_ERR_INVALID_ARG;
    if ((uintptr_t)workspace_dev % 256) return MPT_ERR_WORKSPACE;
    mpt_ctx *c = new (std::nothrow) mpt_ctx();
    if (!c) return MPT_ERR_INTERNAL;
    const int n_states = opt_states(*opt);
    c->use_momentum = n_states >= 1;
    c->opt_kind = opt->kind; c->beta2 = opt->beta2; c->eps = opt->eps; c->wd = opt->weight_decay; c->clip = opt->clip_norm;
    make_plan(layers, n_layers, max_batch, n_states, c->plan, replicas, rank);
    if (workspace_bytes < c->plan.total) { delete c; return MPT_ERR_WORKSPACE; }
    if (replicas > 1) { c->shard_R = replicas; c->shard_rank = rank; }
    const float lr = opt->lr, momentum = opt->momentum;
    c->S = S; c->lr = lr; c->mu = momentum; c->max_batch = max_batch;
    c->stream = (cudaStream_t)cuda_stream;
    c->ws = (uint8_t *)workspace_dev;
    const Plan &pl = c->plan;
    c->status = (uint32_t *)(c->ws + pl.off_status);
    c->master = (float *)(c->ws + pl.off_master) - pl.st_lo;
    c->mom = c->use_momentum ? (float *)(c->ws + pl.off_mom) - pl.st_lo : nullptr;
    c->state2 = n_states >= 2 ? (float *)(c->ws + pl.off_state2) - pl.st_lo : nullptr;
    c->w16 = (uint16_t *)(c->ws + pl.off_w16);
    c->g16 = (uint16_t *)(c->ws + pl.off_g16);
    for (int k = 0; k < 2; k++) {
        c->x_stage[k] = (uint16_t *)(c->ws + pl.off_x[k]);
        c->labels_stage[k] = (int32_t *)(c->ws + pl.off_labels[k]);
    }
    c->row_loss = (float *)(c->ws + pl.off_rowloss);
    c->norm_parts = (double *)(c->ws + pl.off_norm);
    c->splitk_ws = pl.splitk_bytes ? (float *)(c->ws + pl.off_splitk) : nullptr;
    c->layers.resize(n_layers);
    for (int l = 0; l < n_layers; l++) {
        Layer &ly = c->layers[l];
        ly.in = layers[l].in_features; ly.out = layers[l].out_features; ly.relu = layers[l].relu;
        ly.off = pl.lay_off[l];
        ly.n = (size_t)ly.in * ly.out;
        ly.ld_out = pl.ld_out[l];
        ly.act = (uint16_t *)(c->ws + pl.off_act[l]);
        ly.dact = (uint16_t *)(c->ws + pl.off_dact[l]);
    }
    const char *env = getenv("MPT_DISABLE_TC");
    c->disable_tc = env && env[0] == '1';
    env = getenv("MPT_DISABLE_PAIR");
    c->disable_pair = env && env[0] == '1';
    // Parameter arenas (including the padding between layers), activations and status start at zero.
    cudaError_t e = cudaMemsetAsync(c->ws, 0, pl.total, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e == cudaSuccess && push_scale(c) != MPT_OK) e = cudaErrorUnknown;
    if (e == cudaSuccess && push_adam_products(c, 1.0f, 1.0f) != MPT_OK) e = cudaErrorUnknown;
    for (int k = 0; k < 2 && e == cudaSuccess; k++) {
        e = cudaEventCreateWithFlags(&c->staged_ev[k], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->used_ev[k], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) { mpt_destroy(c); return MPT_ERR_CUDA; }
    *out = c;
    return MPT_OK;
}

void mpt_destroy(mpt_ctx *c)
{
    if (!c) return;
    for (auto e : c->ev_own) if (e) cudaEventDestroy(e);
    for (auto &v : c->ev_peer) for (auto e : v) if (e) cudaEventDestroy(e);
    if (c->ev_reduced) cudaEventDestroy(c->ev_reduced);
    if (c->dp_stream) cudaStreamDestroy(c->dp_stream);
    for (auto &sp : c->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (auto &sp : c->pool) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (int k = 0; k < 2; k++) {
        if (c->staged_ev[k]) cudaEventDestroy(c->staged_ev[k]);
        if (c->used_ev[k]) cudaEventDestroy(c->used_ev[k]);
    }
    delete c;
}

int mpt_profile(mpt_ctx *c, int enable)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    for (auto &sp : c->spans) c->pool.push_back(sp);
    c->spans.clear();
    for (int k = 0; k < MPT_PROF_CLASSES; k++) { c->prof_ms[k] = 0; c->prof_work[k] = 0; c->prof_launches[k] = 0; }
    c->profiling = enable != 0;
    return MPT_OK;
}

int mpt_profile_read(mpt_ctx *c, double *ms_out, double *work_out, long long *launches_out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!ms_out || !work_out || !launches_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    for (auto &sp : c->spans) {
        float ms = 0.0f;
        CK(cudaEventElapsedTime(&ms, sp.a, sp.b), "event elapsed time");
        c->prof_ms[sp.cls] += ms;
        c->pool.push_back(sp);
    }
    c->spans.clear();
    for (int k = 0; k < MPT_PROF_CLASSES; k++) {
        ms_out[k] = c->prof_ms[k]; work_out[k] = c->prof_work[k]; launches_out[k] = c->prof_launches[k];
    }
    return MPT_OK;
}

const char *mpt_last_error(mpt_ctx *c) { return c ? c->err.c_str() : "null context"; }

int mpt_launch_count(mpt_ctx *c, long long *count_out)
{
    if (!c || !count_out) return MPT_ERR_INVALID_ARG;
    *count_out = c->launches;
    return MPT_OK;
}

int mpt_set_scale(mpt_ctx *c, float S)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!valid_scale(S)) return fail(c, MPT_ERR_INVALID_ARG, "loss scale out of range");
    c->S = S;
    return push_scale(c);
}

int mpt_get_scale(mpt_ctx *c, float *S_out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!S_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    uint32_t st[ST_WORDS];
    r = read_status(c, st);
    if (r != MPT_OK) return r;
    memcpy(S_out, &st[ST_SCALE], 4);
    c->S = *S_out;
    return MPT_OK;
}

int mpt_set_dynamic_scale(mpt_ctx *c, int enable, int growth_interval, float min_scale, float max_scale)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (enable) {
        if (growth_interval < 1) return fail(c, MPT_ERR_INVALID_ARG, "growth interval must be >= 1");
        if (!valid_scale(min_scale) || !valid_scale(max_scale) || min_scale > max_scale)
            return fail(c, MPT_ERR_INVALID_ARG, "scale bounds out of range");
        c->growth_interval = growth_interval;
        c->scale_min = min_scale;
        c->scale_max = max_scale;
    }
    c->dynamic_scale = enable != 0;
    // the counter of clean steps restarts; S itself is kept (read it back so the host copy is current)
    float S = 0.0f;
    r = mpt_get_scale(c, &S);
    if (r != MPT_OK) return r;
    if (enable) {
        if (S < min_scale) S = min_scale;
        if (S > max_scale) S = max_scale;
    }
    c->S = S;
    return push_scale(c);
}

int mpt_set_lr(mpt_ctx *c, float lr)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!std::isfinite(lr)) return fail(c, MPT_ERR_INVALID_ARG, "learning rate not finite");
    c->lr = lr;
    return MPT_OK;
}

int mpt_set_master(mpt_ctx *c, int layer, const float *src_host, size_t n)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!src_host) return fail(c, MPT_ERR_INVALID_ARG, "null source");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    Layer &ly = c->layers[layer];
    if (n != ly.n) return fail(c, MPT_ERR_SHAPE, "n must equal out*in");
    if (c->shard_R > 1) {
        // FP32 values of the whole layer pass through the gradient array (as scratch, in pieces) to be
        // rounded into the FP16 weights; the part inside the shard is kept as the master copy
        float *scratch = (float *)c->g16;
        const size_t cap = c->plan.P_pad / 2;
        c->have_grads = false;
        for (size_t at = 0; at < n; at += cap) {
            const size_t m = n - at < cap ? n - at : cap;
            CK(cudaMemcpyAsync(scratch, src_host + at, m * 4, cudaMemcpyHostToDevice, c->stream), "master upload");
            cudaError_t e = launch_recast(scratch, c->w16 + ly.off + at, m, c->stream);
            c->launches++;
            if (e != cudaSuccess) return cuda_fail(c, e, "recast launch");
        }
        CK(cudaMemsetAsync(c->g16, 0, c->plan.P_pad * 2, c->stream), "gradient clear");
        size_t first = 0, count = 0;
        state_part(c, ly, &first, &count);
        if (count) CK(cudaMemcpyAsync(c->master + ly.off + first, src_host + first, count * 4, cudaMemcpyHostToDevice, c->stream), "master upload");
        CK(cudaStreamSynchronize(c->stream), "stream synchronize");
        return MPT_OK;
    }
    CK(cudaMemcpyAsync(c->master + ly.off, src_host, n * 4, cudaMemcpyHostToDevice, c->stream), "master upload");
    cudaError_t e = launch_recast(c->master + ly.off, c->w16 + ly.off, n, c->stream);
    c->launches++;
    if (e != cudaSuccess) return cuda_fail(c, e, "recast launch");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int mpt_state_range(mpt_ctx *c, int layer, size_t *first_out, size_t *count_out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!first_out || !count_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    state_part(c, c->layers[layer], first_out, count_out);
    return MPT_OK;
}

int mpt_get_master(mpt_ctx *c, int layer, float *dst_host, size_t n)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!dst_host) return fail(c, MPT_ERR_INVALID_ARG, "null destination");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    Layer &ly = c->layers[layer];
    if (n != ly.n) return fail(c, MPT_ERR_SHAPE, "n must equal out*in");
    size_t first = 0, count = 0;
    state_part(c, ly, &first, &count);
    if (count) CK(cudaMemcpyAsync(dst_host + first, c->master + ly.off + first, count * 4, cudaMemcpyDeviceToHost, c->stream), "master download");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int mpt_forward(mpt_ctx *c, const uint16_t *x_dev, int batch)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!x_dev) return fail(c, MPT_ERR_INVALID_ARG, "null input");
    return do_forward(c, x_dev, batch);
}

int mpt_backward_scaled(mpt_ctx *c, const int32_t *labels_dev, float *loss_host_or_null)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!labels_dev) return fail(c, MPT_ERR_INVALID_ARG, "null labels");
    r = do_backward(c, labels_dev);
    if (r != MPT_OK) return r;
    if (loss_host_or_null) {
        uint32_t st[ST_WORDS];
        r = read_status(c, st);
        if (r != MPT_OK) return r;
        memcpy(loss_host_or_null, &st[ST_LOSS], 4);
        if (st[ST_BAD_LABELS]) return fail(c, MPT_ERR_INVALID_ARG, "labels outside [0, C) were ignored");
    }
    return MPT_OK;
}

int mpt_step(mpt_ctx *c, int *overflow_host_or_null)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    r = do_step(c);
    if (r != MPT_OK) return r;
    if (overflow_host_or_null) {
        uint32_t st[ST_WORDS];
        r = read_status(c, st);
        if (r != MPT_OK) return r;
        return finish_step(c, st, overflow_host_or_null);
    }
    return MPT_OK;
}

int mpt_train_step_host(mpt_ctx *c, const uint16_t *x_host, const int32_t *labels_host, int batch, float *loss_host,
                        int *overflow_host)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!x_host || !labels_host) return fail(c, MPT_ERR_INVALID_ARG, "null host input");
    if (batch < 1 || batch > c->max_batch) return fail(c, MPT_ERR_SHAPE, "batch outside [1, max_batch]");
    if (c->staged_valid[0] || c->staged_valid[1])
        return fail(c, MPT_ERR_STATE, "a staged batch is pending: use mpt_train_step_staged");
    CK(cudaMemcpyAsync(c->x_stage[0], x_host, (size_t)batch * c->layers[0].in * 2, cudaMemcpyHostToDevice, c->stream),
       "input upload");
    CK(cudaMemcpyAsync(c->labels_stage[0], labels_host, (size_t)batch * 4, cudaMemcpyHostToDevice, c->stream), "label upload");
    r = do_forward(c, c->x_stage[0], batch);
    if (r != MPT_OK) return r;
    r = do_backward(c, c->labels_stage[0]);
    if (r != MPT_OK) return r;
    r = do_step(c);
    if (r != MPT_OK) return r;
    uint32_t st[ST_WORDS];
    r = read_status(c, st);
    if (r != MPT_OK) return r;
    if (loss_host) memcpy(loss_host, &st[ST_LOSS], 4);
    r = finish_step(c, st, overflow_host);
    if (r != MPT_OK) return r;
    if (st[ST_BAD_LABELS]) return fail(c, MPT_ERR_INVALID_ARG, "labels outside [0, C) were ignored");
    return MPT_OK;
}

int mpt_stage_batch_host(mpt_ctx *c, const uint16_t *x_host, const int32_t *labels_host, int batch, void *copy_stream)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!x_host || !labels_host) return fail(c, MPT_ERR_INVALID_ARG, "null host input");
    if (batch < 1 || batch > c->max_batch) return fail(c, MPT_ERR_SHAPE, "batch outside [1, max_batch]");
    const int k = c->stage_w;
    if (c->staged_valid[k]) return fail(c, MPT_ERR_STATE, "both staging slots hold unconsumed batches");
    cudaStream_t cs = (cudaStream_t)copy_stream;
    // the slot's previous consumer (the step that read it) must have finished before it is overwritten
    if (c->used_recorded[k]) CK(cudaStreamWaitEvent(cs, c->used_ev[k], 0), "wait for the slot's last consumer");
    CK(cudaMemcpyAsync(c->x_stage[k], x_host, (size_t)batch * c->layers[0].in * 2, cudaMemcpyHostToDevice, cs), "input upload");
    CK(cudaMemcpyAsync(c->labels_stage[k], labels_host, (size_t)batch * 4, cudaMemcpyHostToDevice, cs), "label upload");
    CK(cudaEventRecord(c->staged_ev[k], cs), "event record");
    c->staged_valid[k] = true;
    c->staged_batch[k] = batch;
    c->stage_w ^= 1;
    return MPT_OK;
}

int mpt_train_step_staged(mpt_ctx *c, float *loss_host, int *overflow_host)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    const int k = c->stage_r;
    if (!c->staged_valid[k]) return fail(c, MPT_ERR_STATE, "no staged batch: call mpt_stage_batch_host first");
    CK(cudaStreamWaitEvent(c->stream, c->staged_ev[k], 0), "wait for the staged batch");
    r = do_forward(c, c->x_stage[k], c->staged_batch[k]);
    if (r != MPT_OK) return r;
    r = do_backward(c, c->labels_stage[k]);
    if (r != MPT_OK) return r;
    r = do_step(c);
    if (r != MPT_OK) return r;
    CK(cudaEventRecord(c->used_ev[k], c->stream), "event record");
    c->used_recorded[k] = true;
    c->staged_valid[k] = false;
    c->stage_r ^= 1;
    uint32_t st[ST_WORDS];
    r = read_status(c, st);
    if (r != MPT_OK) return r;
    if (loss_host) memcpy(loss_host, &st[ST_LOSS], 4);
    r = finish_step(c, st, overflow_host);
    if (r != MPT_OK) return r;
    if (st[ST_BAD_LABELS]) return fail(c, MPT_ERR_INVALID_ARG, "labels outside [0, C) were ignored");
    return MPT_OK;
}

int mpt_get_tensor(mpt_ctx *c, int kind, int layer, void *dst_host, size_t bytes)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!dst_host) return fail(c, MPT_ERR_INVALID_ARG, "null destination");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    Layer &ly = c->layers[layer];
    const void *src = nullptr;
    size_t rows = 0, row_bytes = 0, pitch = 0;
    switch (kind) {
        case MPT_T_W16: src = c->w16 + ly.off; rows = 1; row_bytes = ly.n * 2; pitch = row_bytes; break;
        case MPT_T_GRAD16: src = c->g16 + ly.off; rows = 1; row_bytes = ly.n * 2; pitch = row_bytes; break;
        case MPT_T_MASTER32: src = c->master + ly.off; rows = 1; row_bytes = ly.n * 4; pitch = row_bytes; break;
        case MPT_T_MOMENTUM32:
            if (!c->use_momentum) return fail(c, MPT_ERR_STATE, "context has no momentum buffer");
            src = c->mom + ly.off; rows = 1; row_bytes = ly.n * 4; pitch = row_bytes; break;
        case MPT_T_STATE2_32:
            if (!c->state2) return fail(c, MPT_ERR_STATE, "context has no second optimizer state");
            src = c->state2 + ly.off; rows = 1; row_bytes = ly.n * 4; pitch = row_bytes; break;
        case MPT_T_ACT16:
        case MPT_T_DACT16:
            if (c->batch < 1) return fail(c, MPT_ERR_STATE, "no forward pass yet");
            src = kind == MPT_T_ACT16 ? ly.act : ly.dact;
            rows = (size_t)c->batch; row_bytes = (size_t)ly.out * 2; pitch = (size_t)ly.ld_out * 2; break;
        default: return fail(c, MPT_ERR_INVALID_ARG, "tensor kind");
    }
    if (bytes != rows * row_bytes) return fail(c, MPT_ERR_SHAPE, "byte count does not match the tensor");
    if (c->shard_R > 1 && (kind == MPT_T_MASTER32 || kind == MPT_T_MOMENTUM32 || kind == MPT_T_STATE2_32)) {
        // only the part inside this replica's shard exists (mpt_state_range); the rest of dst_host is left alone
        size_t first = 0, count = 0;
        state_part(c, ly, &first, &count);
        if (count) CK(cudaMemcpyAsync((float *)dst_host + first, (const float *)src + first, count * 4, cudaMemcpyDeviceToHost, c->stream), "tensor download");
        CK(cudaStreamSynchronize(c->stream), "stream synchronize");
        return MPT_OK;
    }
    CK(cudaMemcpy2DAsync(dst_host, row_bytes, src, pitch, row_bytes, rows, cudaMemcpyDeviceToHost, c->stream), "tensor download");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int mpt_set_grad(mpt_ctx *c, int layer, const uint16_t *src_host, size_t n)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!src_host) return fail(c, MPT_ERR_INVALID_ARG, "null source");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    Layer &ly = c->layers[layer];
    if (n != ly.n) return fail(c, MPT_ERR_SHAPE, "n must equal out*in");
    CK(cudaMemcpyAsync(c->g16 + ly.off, src_host, n * 2, cudaMemcpyHostToDevice, c->stream), "gradient upload");
    // the overflow word must describe all layers' gradients as they now stand
    CK(cudaMemsetAsync(c->status + ST_OVERFLOW, 0, sizeof(uint32_t), c->stream), "status clear");
    cudaError_t e = launch_grad_nonfinite(c->g16, c->plan.P_pad, 1.0f / c->S, c->status + ST_OVERFLOW, c->stream);
    c->launches++;
    if (e != cudaSuccess) return cuda_fail(c, e, "inspection launch");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    c->have_grads = true;
    return MPT_OK;
}

int mpt_set_momentum(mpt_ctx *c, int layer, const float *src_host, size_t n)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!src_host) return fail(c, MPT_ERR_INVALID_ARG, "null source");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    if (!c->use_momentum) return fail(c, MPT_ERR_STATE, "context has no momentum buffer");
    Layer &ly = c->layers[layer];
    if (n != ly.n) return fail(c, MPT_ERR_SHAPE, "n must equal out*in");
    size_t first = 0, count = 0;
    state_part(c, ly, &first, &count);
    if (count) CK(cudaMemcpyAsync(c->mom + ly.off + first, src_host + first, count * 4, cudaMemcpyHostToDevice, c->stream), "momentum upload");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int mpt_set_state2(mpt_ctx *c, int layer, const float *src_host, size_t n)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!src_host) return fail(c, MPT_ERR_INVALID_ARG, "null source");
    if (layer < 0 || layer >= (int)c->layers.size()) return fail(c, MPT_ERR_INVALID_ARG, "layer index");
    if (!c->state2) return fail(c, MPT_ERR_STATE, "context has no second optimizer state");
    Layer &ly = c->layers[layer];
    if (n != ly.n) return fail(c, MPT_ERR_SHAPE, "n must equal out*in");
    size_t first = 0, count = 0;
    state_part(c, ly, &first, &count);
    if (count) CK(cudaMemcpyAsync(c->state2 + ly.off + first, src_host + first, count * 4, cudaMemcpyHostToDevice, c->stream), "state upload");
    CK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int mpt_get_adam_products(mpt_ctx *c, float *b1t_out, float *b2t_out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!b1t_out || !b2t_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    uint32_t st[ST_WORDS];
    r = read_status(c, st);
    if (r != MPT_OK) return r;
    memcpy(b1t_out, &st[ST_B1T], 4);
    memcpy(b2t_out, &st[ST_B2T], 4);
    return MPT_OK;
}

int mpt_get_grad_norm(mpt_ctx *c, float *norm_out, float *coef_out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!norm_out || !coef_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    if (c->clip <= 0.0f) return fail(c, MPT_ERR_STATE, "the context was created without gradient clipping");
    uint32_t st[ST_WORDS];
    r = read_status(c, st);
    if (r != MPT_OK) return r;
    memcpy(norm_out, &st[ST_GRAD_NORM], 4);
    memcpy(coef_out, &st[ST_CLIP_COEF], 4);
    return MPT_OK;
}

int mpt_dp_layout_of(mpt_ctx *c, mpt_dp_layout *out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    out->g16_offset = (size_t)((const uint8_t *)c->g16 - c->ws);
    out->w16_offset = (size_t)((const uint8_t *)c->w16 - c->ws);
    out->flags_offset = (size_t)((const uint8_t *)(c->status + ST_OVERFLOW) - c->ws);
    out->n = c->plan.P_pad;
    return MPT_OK;
}

int mpt_dp_attach(mpt_ctx *c, int R, int rank, const uint16_t *const *g16_peers, const uint32_t *const *flag_peers,
                  uint16_t *const *w16_peers)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (R == 1) {
        c->dp_R = 0;
        return MPT_OK;
    }
    if (R < 2 || R > MPT_DP_MAX_REPLICAS || rank < 0 || rank >= R) return fail(c, MPT_ERR_INVALID_ARG, "replica count or rank");
    if (c->shard_R > 1 && (R != c->shard_R || rank != c->shard_rank))
        return fail(c, MPT_ERR_INVALID_ARG, "the context was created by mpt_create_dp for another replica count or rank");
    if (!g16_peers || !flag_peers || !w16_peers) return fail(c, MPT_ERR_INVALID_ARG, "null peer table");
    for (int q = 0; q < R; q++) {
        if (!g16_peers[q] || !flag_peers[q] || !w16_peers[q]) return fail(c, MPT_ERR_INVALID_ARG, "null peer pointer");
        if ((((uintptr_t)g16_peers[q] | (uintptr_t)w16_peers[q]) & 15) != 0 || ((uintptr_t)flag_peers[q] & 3) != 0)
            return fail(c, MPT_ERR_INVALID_ARG, "misaligned peer pointer");
    }
    if (g16_peers[rank] != c->g16 || w16_peers[rank] != c->w16 || flag_peers[rank] != c->status + ST_OVERFLOW)
        return fail(c, MPT_ERR_INVALID_ARG, "this replica's entries must be the context's own buffers");
    for (int q = 0; q < R; q++) {
        c->dp_g16[q] = g16_peers[q];
        c->dp_flag[q] = flag_peers[q];
        c->dp_w16[q] = w16_peers[q];
    }
    c->dp_R = R;
    c->dp_rank = rank;
    return MPT_OK;
}

int mpt_dp_norm(mpt_ctx *c)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (c->dp_R < 2) return fail(c, MPT_ERR_STATE, "mpt_dp_norm needs an attached data-parallel context");
    if (c->clip <= 0.0f) return fail(c, MPT_ERR_STATE, "the context was created without gradient clipping");
    if (!c->have_grads) return fail(c, MPT_ERR_STATE, "mpt_dp_norm needs gradients (mpt_backward_scaled or mpt_set_grad)");
    size_t lo = 0, hi = 0;
    mpt_dp_shard(c->plan.P_pad, c->dp_R, c->dp_rank, &lo, &hi);
    const float inv_SR = 1.0f / (c->S * (float)c->dp_R);
    cudaError_t e = launch_dp_sqnorm(c->dp_g16, c->dp_R, lo, hi - lo, inv_SR, (const float *)(c->status + ST_SCALE), c->norm_parts,
                                     (double *)(c->status + ST_DP_NORM), c->stream);
    c->launches += 2;
    if (e != cudaSuccess) return cuda_fail(c, e, "data-parallel norm launch");
    c->dp_norm_done = true;
    return MPT_OK;
}

int mpt_dp_overlap_events(mpt_ctx *c, uint8_t *handles_out)
{
    static_assert(sizeof(cudaIpcEventHandle_t) == MPT_DP_HANDLE_BYTES, "handle size");
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!handles_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    const size_t L = c->layers.size() + 1;      // one per layer and one for the published norm (clipping)
    if (c->ev_own.empty()) {
        c->ev_own.resize(L, nullptr);
        for (size_t l = 0; l < L; l++)
            CK(cudaEventCreateWithFlags(&c->ev_own[l], cudaEventDisableTiming | cudaEventInterprocess), "event create");
    }
    for (size_t l = 0; l < L; l++) {
        cudaIpcEventHandle_t h;
        CK(cudaIpcGetEventHandle(&h, c->ev_own[l]), "event export");
        memcpy(handles_out + l * MPT_DP_HANDLE_BYTES, &h, MPT_DP_HANDLE_BYTES);
    }
    return MPT_OK;
}

int mpt_dp_overlap_attach(mpt_ctx *c, const uint8_t *const *peer_handles, float *sum32_dev, size_t sum32_bytes)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (c->dp_R < 2) return fail(c, MPT_ERR_STATE, "mpt_dp_overlap_attach needs an attached data-parallel context");
    if (c->ev_own.empty()) return fail(c, MPT_ERR_STATE, "call mpt_dp_overlap_events first");
    if (c->dp_overlap) return fail(c, MPT_ERR_STATE, "already attached");
    if (!peer_handles || !sum32_dev) return fail(c, MPT_ERR_INVALID_ARG, "null argument");
    size_t lo = 0, hi = 0;
    mpt_dp_shard(c->plan.P_pad, c->dp_R, c->dp_rank, &lo, &hi);
    if (sum32_bytes < (hi - lo) * 4 || ((uintptr_t)sum32_dev & 15)) return fail(c, MPT_ERR_WORKSPACE, "scratch for the sums too small or misaligned");
    const size_t L = c->layers.size() + 1;
    for (int q = 0; q < c->dp_R; q++) {
        if (q == c->dp_rank) continue;
        if (!peer_handles[q]) return fail(c, MPT_ERR_INVALID_ARG, "null peer handles");
        c->ev_peer[q].assign(L, nullptr);
        for (size_t l = 0; l < L; l++) {
            cudaIpcEventHandle_t h;
            memcpy(&h, peer_handles[q] + l * MPT_DP_HANDLE_BYTES, MPT_DP_HANDLE_BYTES);
            CK(cudaIpcOpenEventHandle(&c->ev_peer[q][l], h), "event open");
        }
    }
    CK(cudaStreamCreateWithFlags(&c->dp_stream, cudaStreamNonBlocking), "stream create");
    CK(cudaEventCreateWithFlags(&c->ev_reduced, cudaEventDisableTiming), "event create");
    c->sum32 = sum32_dev;
    c->dp_overlap = true;
    c->dp_reduced = false;
    return MPT_OK;
}

int mpt_dp_reduce_async(mpt_ctx *c)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!c->dp_overlap) return fail(c, MPT_ERR_STATE, "mpt_dp_reduce_async needs mpt_dp_overlap_attach");
    if (!c->have_grads) return fail(c, MPT_ERR_STATE, "mpt_dp_reduce_async needs gradients (mpt_backward_scaled or mpt_set_grad)");
    size_t lo = 0, hi = 0;
    mpt_dp_shard(c->plan.P_pad, c->dp_R, c->dp_rank, &lo, &hi);
    const int L = (int)c->layers.size();
    for (int l = L - 1; l >= 0; l--) {      // the order in which the backward pass completes the layers
        const size_t a0 = c->layers[l].off, b0 = l + 1 < L ? c->layers[l + 1].off : c->plan.P_pad;   // with the padding after it
        const size_t a = a0 > lo ? a0 : lo, b = b0 < hi ? b0 : hi;
        if (a >= b) continue;
        for (int q = 0; q < c->dp_R; q++)
            CK(cudaStreamWaitEvent(c->dp_stream, q == c->dp_rank ? c->ev_own[l] : c->ev_peer[q][l], 0), "event wait");
        cudaError_t e = launch_dp_reduce(c->dp_g16, c->dp_R, a, b - a, c->sum32 + (a - lo), c->dp_stream);
        c->launches++;
        if (e != cudaSuccess) return cuda_fail(c, e, "reduce launch");
    }
    if (c->clip > 0.0f) {
        // this replica's part of the squared norm of the mean gradient, from the sums, published next to its
        // overflow word; the event tells the other replicas when it is there
        const float inv_SR = 1.0f / (c->S * (float)c->dp_R);
        cudaError_t e = launch_dp_sqnorm(c->dp_g16, c->dp_R, lo, hi - lo, inv_SR, (const float *)(c->status + ST_SCALE), c->norm_parts,
                                         (double *)(c->status + ST_DP_NORM), c->dp_stream, c->sum32);
        c->launches += 2;
        if (e != cudaSuccess) return cuda_fail(c, e, "norm launch");
        CK(cudaEventRecord(c->ev_own[L], c->dp_stream), "event record");
        c->dp_norm_done = true;
    }
    CK(cudaEventRecord(c->ev_reduced, c->dp_stream), "event record");
    c->dp_reduced = true;
    return MPT_OK;
}

int mpt_set_adam_products(mpt_ctx *c, float b1t, float b2t)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!std::isfinite(b1t) || !std::isfinite(b2t)) return fail(c, MPT_ERR_INVALID_ARG, "products must be finite");
    return push_adam_products(c, b1t, b2t);
}

// ---------------------------------------------------------- stateless launchers

int mpt_gemm_workspace_bytes(int op, int M, int N, int K, size_t *bytes_out)
{
    if (!bytes_out) return MPT_ERR_INVALID_ARG;
    if (op != MPT_OP_FWD && op != MPT_OP_DGRAD && op != MPT_OP_WGRAD) return MPT_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || K < 0) return MPT_ERR_SHAPE;
    *bytes_out = 0;
    if (M == 0 || N == 0 || K == 0) return MPT_OK;
    if (tc4_split_for(M, N, K)) return MPT_OK;       // the in-cluster split needs no scratch
    tc_choose_pair(M, N, K, (size_t)256 << 20, bytes_out);
    return MPT_OK;
}

int mpt_gemm_f16(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb, uint16_t *C, int ldc,
                 unsigned flags, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag, uint32_t *status_dev,
                 void *cuda_stream)
{
    return mpt_gemm_f16_ws(op, M, N, K, A, lda, B, ldb, C, ldc, flags, mask, ldmask, nonfinite_flag, status_dev, nullptr, 0,
                           cuda_stream);
}

int mpt_gemm_f16_ws(int op, int M, int N, int K, const uint16_t *A, int lda, const uint16_t *B, int ldb, uint16_t *C,
                    int ldc, unsigned flags, const uint16_t *mask, int ldmask, uint32_t *nonfinite_flag,
                    uint32_t *status_dev, void *splitk_ws_dev, size_t splitk_ws_bytes, void *cuda_stream)
{
    return mpt::dispatch_gemm(op, M, N, K, A, lda, B, ldb, C, ldc, flags, mask, ldmask, nonfinite_flag, status_dev,
                              splitk_ws_dev, splitk_ws_bytes, (cudaStream_t)cuda_stream, nullptr);
}

int mpt_recast(const float *w32_dev, uint16_t *w16_dev, size_t n, void *cuda_stream)
{
    if (!w32_dev || !w16_dev) return MPT_ERR_INVALID_ARG;
    return launch_recast(w32_dev, w16_dev, n, (cudaStream_t)cuda_stream) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_grad_nonfinite(const uint16_t *g16_dev, size_t n, float inv_S, uint32_t *flag_dev, void *cuda_stream)
{
    if (!g16_dev || !flag_dev) return MPT_ERR_INVALID_ARG;
    return launch_grad_nonfinite(g16_dev, n, inv_S, flag_dev, (cudaStream_t)cuda_stream) == cudaSuccess ? MPT_OK
                                                                                                       : MPT_ERR_CUDA;
}

int mpt_update_flat(const uint16_t *g16_dev, float *w32_dev, float *v_dev, uint16_t *w16_dev, size_t n, float inv_S,
                    float lr, float mu, int use_momentum, int detect, uint32_t *flags_dev, void *cuda_stream)
{
    if (!g16_dev || !w32_dev || !w16_dev || !flags_dev) return MPT_ERR_INVALID_ARG;
    if (use_momentum && !v_dev) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (detect) {
        e = cudaMemsetAsync(flags_dev, 0, 2 * sizeof(uint32_t), st);
        if (e == cudaSuccess) e = launch_grad_nonfinite(g16_dev, n, inv_S, flags_dev, st);
    } else {
        e = cudaMemsetAsync(flags_dev + 1, 0, sizeof(uint32_t), st);
    }
    if (e == cudaSuccess) e = launch_update(g16_dev, w32_dev, v_dev, w16_dev, n, inv_S, lr, mu, use_momentum != 0, flags_dev, st);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_update_flat_opt(const mpt_optimizer *opt, const uint16_t *g16_dev, float *w32_dev, float *s1_dev, float *s2_dev,
                        uint16_t *w16_dev, size_t n, float inv_S, float b1t, float b2t, int detect, uint32_t *flags_dev,
                        void *clip_scratch_dev, void *cuda_stream)
{
    if (!g16_dev || !w32_dev || !w16_dev || !flags_dev) return MPT_ERR_INVALID_ARG;
    if (!valid_optimizer(opt)) return MPT_ERR_INVALID_ARG;
    const bool clip = opt->clip_norm > 0.0f;
    if (clip && (!clip_scratch_dev || ((uintptr_t)clip_scratch_dev & 255) != 0)) return MPT_ERR_INVALID_ARG;
    const int ns = opt_states(*opt);
    if ((ns >= 1 && !s1_dev) || (ns >= 2 && !s2_dev)) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (detect) {
        e = cudaMemsetAsync(flags_dev, 0, 2 * sizeof(uint32_t), st);
        if (e == cudaSuccess) e = launch_grad_nonfinite(g16_dev, n, inv_S, flags_dev, st);
    } else {
        e = cudaMemsetAsync(flags_dev + 1, 0, sizeof(uint32_t), st);
    }
    float *coef_dev = nullptr;
    if (e == cudaSuccess && clip) {   // scratch: two floats (coefficient, norm), then the partial sums at byte 256
        coef_dev = (float *)clip_scratch_dev;
        e = launch_clip_coef(g16_dev, n, inv_S, nullptr, opt->clip_norm, (double *)((char *)clip_scratch_dev + 256), coef_dev, st);
    }
    if (e == cudaSuccess)
        e = launch_update_opt(opt->kind, g16_dev, w32_dev, ns >= 1 ? s1_dev : nullptr, ns >= 2 ? s2_dev : nullptr, w16_dev, n,
                              inv_S, opt->lr, opt->momentum, opt->beta2, opt->eps, opt->weight_decay, b1t, b2t, flags_dev, st,
                              nullptr, nullptr, coef_dev);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_softmax_ce(const uint16_t *z_dev, int ldz, const int32_t *labels_dev, int B, int C, float S, uint16_t *dz_dev,
                   int lddz, float *row_loss_dev, float *loss_dev, uint32_t *bad_labels_dev, uint32_t *status_dev,
                   void *cuda_stream)
{
    if (!z_dev || !labels_dev || !dz_dev || !row_loss_dev || !loss_dev) return MPT_ERR_INVALID_ARG;
    if (B < 0 || C < 0 || ldz < C || lddz < C) return MPT_ERR_SHAPE;
    if (z_dev == dz_dev) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaSuccess;
    if (bad_labels_dev) e = cudaMemsetAsync(bad_labels_dev, 0, sizeof(uint32_t), st);
    if (e == cudaSuccess)
        e = launch_softmax_ce(z_dev, ldz, labels_dev, B, C, S, dz_dev, lddz, row_loss_dev, loss_dev, bad_labels_dev, st, nullptr,
                              nullptr, status_dev);
    return e == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_sm_clock_probe(unsigned window_us, float *mhz_dev, void *cuda_stream)
{
    if (!mhz_dev) return MPT_ERR_INVALID_ARG;
    if (window_us < 1 || window_us > 100000u) return MPT_ERR_INVALID_ARG;
    return launch_clock_probe(window_us, mhz_dev, (cudaStream_t)cuda_stream) == cudaSuccess ? MPT_OK : MPT_ERR_CUDA;
}

int mpt_selftest_wait_timeout(unsigned limit_us, uint32_t *status_dev, void *cuda_stream)
{
    if (!status_dev) return MPT_ERR_INVALID_ARG;
    if (limit_us < 1 || limit_us > 2000000u) return MPT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (launch_wait_selftest(limit_us, status_dev, st) != cudaSuccess) return MPT_ERR_CUDA;
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, status_dev, sizeof word, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MPT_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return MPT_ERR_CUDA;
    return word != 0 ? MPT_ERR_TIMEOUT : MPT_OK;
}

int mpt_selftest_wait_timeout_ctx(mpt_ctx *c, unsigned limit_us)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (limit_us < 1 || limit_us > 2000000u) return fail(c, MPT_ERR_INVALID_ARG, "limit outside [1, 2000000] microseconds");
    CK(launch_wait_selftest(limit_us, c->status + ST_KERNEL_ERR, c->stream), "self-test launch");
    c->launches++;
    uint32_t st[ST_WORDS];
    return read_status(c, st);       // MPT_ERR_TIMEOUT, and the context is poisoned from here on
}

}  // extern "C"

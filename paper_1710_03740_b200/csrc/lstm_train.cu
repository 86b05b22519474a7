// A trained LSTM layer with projection (paper section 4.5: the language model's recurrent layer,
// loss scale 128 there, Adagrad): FP32 master copies of Wg, Wp and the bias, FP16 working copies,
// T steps forward, softmax cross-entropy on the projected outputs r_t taken as logits (scaled by
// S, section 3.2), back-propagation through time, overflow inspection riding on the three gradient
// epilogues, optional dynamic loss scale, and the optimizer step on the master copy (section 3.1).
// Host sequencing only: every arithmetic step is a kernel of this library on the caller's stream.
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <string>

#include "mpt_common.cuh"

using namespace mpt;

struct mpt_lstm_ctx {
    mpt_lstm_desc d;
    mpt_lstm_tensors t;
    mpt_optimizer opt;
    int n_states;
    float S;
    cudaStream_t stream;
    uint8_t *ws;
    uint32_t *status;
    float *master, *s1, *s2;
    uint16_t *w16, *g16;
    float *row_loss;
    double *norm_parts;
    size_t off_Wg, off_Wp, off_b, n_total;     // element offsets inside the flat parameter arenas
    size_t total_bytes;
    bool dynamic_scale = false;
    int growth_interval = 2000;
    float scale_min = 0x1p-100f, scale_max = 0x1p120f;
    bool params_set = false, poisoned = false;
    std::string err;
};

namespace {

size_t pad128(size_t n) { return (n + 127) / 128 * 128; }

struct LstmPlan {
    size_t off_status, off_lstatus, off_master, off_s1, off_s2, off_w16, off_g16, off_xr, off_c, off_h, off_acts, off_drext,
        off_dxr, off_drtot, off_dG, off_dh, off_dc, off_bparts, off_rowloss, off_norm, off_splitk, splitk_bytes, total;
    size_t off_Wg, off_Wp, off_b, n_total;
};

void make_plan(const mpt_lstm_desc &d, int n_states, LstmPlan &p)
{
    const size_t T = d.T, B = d.B, I = d.I, H = d.H, P = d.P, K = I + P;
    p.off_Wg = 0;
    p.off_Wp = pad128(4 * H * K);
    p.off_b = p.off_Wp + pad128(P * H);
    p.n_total = p.off_b + pad128(4 * H);
    size_t cur = 0;
    auto take = [&](size_t bytes) { size_t o = cur; cur += (bytes + 255) / 256 * 256; return o; };
    p.off_status = take(ST_WORDS * 4);
    p.off_lstatus = take(16 * 4);
    p.off_master = take(p.n_total * 4);
    p.off_s1 = n_states >= 1 ? take(p.n_total * 4) : 0;
    p.off_s2 = n_states >= 2 ? take(p.n_total * 4) : 0;
    p.off_w16 = take(p.n_total * 2);
    p.off_g16 = take(p.n_total * 2);
    p.off_xr = take((T + 1) * B * K * 2);
    p.off_c = take((T + 1) * B * H * 2);
    p.off_h = take(T * B * H * 2);
    p.off_acts = take(T * B * 4 * H * 2);
    p.off_drext = take(T * B * P * 2);
    p.off_dxr = take(T * B * K * 2);
    p.off_drtot = take(T * B * P * 2);
    p.off_dG = take(T * B * 4 * H * 2);
    p.off_dh = take(B * H * 2);
    p.off_dc = take(2 * B * H * 2);
    p.off_bparts = take((size_t)kBiasRowParts * 4 * H * 4);
    p.off_rowloss = take(T * B * 4);
    p.off_norm = take((size_t)kNormParts * 8);
    size_t need = 0;
    tc_choose_pair((int)B, (int)P, (int)H, (size_t)256 << 20, &need);      // the projection product may split its contraction
    p.splitk_bytes = need;
    p.off_splitk = need ? take(need) : 0;
    p.total = cur;
}

bool valid_desc(const mpt_lstm_desc *d)
{
    if (!d) return false;
    if (d->T < 1 || d->B < 1 || d->I < 8 || d->H < 8 || d->P < 8) return false;
    if ((d->I % 8) || (d->H % 8) || (d->P % 8)) return false;
    if ((long long)d->H * 4 > 0x7FFFFFF0ll || (long long)d->T * d->B > 0x7FFFFFF0ll) return false;
    return true;
}

bool valid_opt(const mpt_optimizer *o)
{
    if (!o) return false;
    if (o->kind < MPT_OPT_SGD || o->kind > MPT_OPT_ADAM) return false;
    if (!isfinite(o->lr) || !(o->momentum >= 0.0f && o->momentum < 1.0f)) return false;
    if (!(o->weight_decay >= 0.0f) || !isfinite(o->weight_decay) || !(o->clip_norm >= 0.0f) || !isfinite(o->clip_norm)) return false;
    if (o->kind == MPT_OPT_ADAM && !(o->beta2 >= 0.0f && o->beta2 < 1.0f)) return false;
    if ((o->kind == MPT_OPT_ADAM || o->kind == MPT_OPT_ADAGRAD) && (!(o->eps >= 0.0f) || !isfinite(o->eps))) return false;
    return true;
}

int states_of(const mpt_optimizer &o)
{
    if (o.kind == MPT_OPT_SGD) return o.momentum != 0.0f ? 1 : 0;
    return o.kind == MPT_OPT_ADAM ? 2 : 1;
}

bool valid_scale(float S) { return isfinite(S) && S >= 0x1p-100f && S <= 0x1p120f; }

int fail(mpt_lstm_ctx *c, int code, const char *msg)
{
    c->err = msg;
    if (code == MPT_ERR_CUDA || code == MPT_ERR_TIMEOUT) c->poisoned = true;
    return code;
}

int cuda_fail(mpt_lstm_ctx *c, cudaError_t e, const char *what)
{
    char buf[256];
    snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
    c->err = buf;
    c->poisoned = true;
    return MPT_ERR_CUDA;
}

#define LCK(call, what)                                         \
    do {                                                        \
        cudaError_t e__ = (call);                               \
        if (e__ != cudaSuccess) return cuda_fail(c, e__, what); \
    } while (0)

int usable(mpt_lstm_ctx *c)
{
    if (!c) return MPT_ERR_INVALID_ARG;
    return c->poisoned ? MPT_ERR_STATE : MPT_OK;
}

int push_scale(mpt_lstm_ctx *c)
{
    uint32_t w[3];
    const float inv = 1.0f / c->S;
    memcpy(&w[0], &c->S, 4);
    memcpy(&w[1], &inv, 4);
    w[2] = 0;
    LCK(cudaMemcpyAsync(c->status + ST_SCALE, w, sizeof w, cudaMemcpyHostToDevice, c->stream), "scale upload");
    LCK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int read_status(mpt_lstm_ctx *c, uint32_t (&st)[ST_WORDS], uint32_t *lstm_err)
{
    LCK(cudaMemcpyAsync(st, c->status, sizeof st, cudaMemcpyDeviceToHost, c->stream), "status copy");
    uint32_t ls[4] = {0, 0, 0, 0};
    LCK(cudaMemcpyAsync(ls, c->t.status_dev, sizeof ls, cudaMemcpyDeviceToHost, c->stream), "status copy");
    LCK(cudaStreamSynchronize(c->stream), "stream synchronize");
    if (lstm_err) *lstm_err = ls[0];
    if (st[ST_KERNEL_ERR] != 0 || ls[0] != 0) return fail(c, MPT_ERR_TIMEOUT, "a device-side bounded wait expired");
    return MPT_OK;
}

}  // namespace

extern "C" {

int mpt_lstm_workspace_bytes(const mpt_lstm_desc *desc, const mpt_optimizer *opt, size_t *bytes_out)
{
    if (!bytes_out || !desc || !opt) return MPT_ERR_INVALID_ARG;
    if (!valid_desc(desc)) return MPT_ERR_SHAPE;
    if (!valid_opt(opt)) return MPT_ERR_INVALID_ARG;
    LstmPlan p;
    make_plan(*desc, states_of(*opt), p);
    *bytes_out = p.total;
    return MPT_OK;
}

int mpt_lstm_create(const mpt_lstm_desc *desc, float S, const mpt_optimizer *opt, void *workspace_dev, size_t workspace_bytes,
                    void *cuda_stream, mpt_lstm_ctx **out)
{
    if (!out) return MPT_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc || !opt || !workspace_dev) return MPT_ERR_INVALID_ARG;
    if (!valid_desc(desc)) return MPT_ERR_SHAPE;
    if (!valid_opt(opt) || !valid_scale(S)) return MPT_ERR_INVALID_ARG;
    if ((uintptr_t)workspace_dev % 256) return MPT_ERR_WORKSPACE;
    LstmPlan p;
    const int ns = states_of(*opt);
    make_plan(*desc, ns, p);
    if (workspace_bytes < p.total) return MPT_ERR_WORKSPACE;
    mpt_lstm_ctx *c = new (std::nothrow) mpt_lstm_ctx();
    if (!c) return MPT_ERR_INTERNAL;
    c->d = *desc;
    c->opt = *opt;
    c->n_states = ns;
    c->S = S;
    c->stream = (cudaStream_t)cuda_stream;
    c->ws = (uint8_t *)workspace_dev;
    c->total_bytes = p.total;
    c->status = (uint32_t *)(c->ws + p.off_status);
    c->master = (float *)(c->ws + p.off_master);
    c->s1 = ns >= 1 ? (float *)(c->ws + p.off_s1) : nullptr;
    c->s2 = ns >= 2 ? (float *)(c->ws + p.off_s2) : nullptr;
    c->w16 = (uint16_t *)(c->ws + p.off_w16);
    c->g16 = (uint16_t *)(c->ws + p.off_g16);
    c->row_loss = (float *)(c->ws + p.off_rowloss);
    c->norm_parts = (double *)(c->ws + p.off_norm);
    c->off_Wg = p.off_Wg; c->off_Wp = p.off_Wp; c->off_b = p.off_b; c->n_total = p.n_total;
    mpt_lstm_tensors &t = c->t;
    memset(&t, 0, sizeof t);
    t.Wg16 = c->w16 + p.off_Wg;
    t.Wp16 = c->w16 + p.off_Wp;
    t.bias16 = c->w16 + p.off_b;
    t.xr = (uint16_t *)(c->ws + p.off_xr);
    t.c = (uint16_t *)(c->ws + p.off_c);
    t.h = (uint16_t *)(c->ws + p.off_h);
    t.acts = (uint16_t *)(c->ws + p.off_acts);
    t.dr_ext = (uint16_t *)(c->ws + p.off_drext);
    t.dxr = (uint16_t *)(c->ws + p.off_dxr);
    t.drtot = (uint16_t *)(c->ws + p.off_drtot);
    t.dG = (uint16_t *)(c->ws + p.off_dG);
    t.dh = (uint16_t *)(c->ws + p.off_dh);
    t.dc = (uint16_t *)(c->ws + p.off_dc);
    t.dWg16 = c->g16 + p.off_Wg;
    t.dWp16 = c->g16 + p.off_Wp;
    t.dbias16 = c->g16 + p.off_b;
    t.bias_parts = (float *)(c->ws + p.off_bparts);
    t.nonfinite_flag = c->status + ST_OVERFLOW;
    t.status_dev = (uint32_t *)(c->ws + p.off_lstatus);
    t.splitk_ws = p.splitk_bytes ? (void *)(c->ws + p.off_splitk) : nullptr;
    t.splitk_ws_bytes = p.splitk_bytes;
    // parameter arenas (with the padding between tensors), recurrent state and status start at zero
    cudaError_t e = cudaMemsetAsync(c->ws, 0, p.total, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e == cudaSuccess && push_scale(c) != MPT_OK) e = cudaErrorUnknown;
    if (e == cudaSuccess) {
        const float one[2] = {1.0f, 1.0f};
        e = cudaMemcpyAsync(c->status + ST_B1T, one, sizeof one, cudaMemcpyHostToDevice, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    }
    if (e != cudaSuccess) { delete c; return MPT_ERR_CUDA; }
    *out = c;
    return MPT_OK;
}

void mpt_lstm_destroy(mpt_lstm_ctx *c) { delete c; }

const char *mpt_lstm_last_error(mpt_lstm_ctx *c) { return c ? c->err.c_str() : "null context"; }

int mpt_lstm_set_params(mpt_lstm_ctx *c, const float *Wg_host, const float *bias_host, const float *Wp_host)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!Wg_host || !bias_host || !Wp_host) return fail(c, MPT_ERR_INVALID_ARG, "null parameter array");
    const size_t H = c->d.H, K = (size_t)c->d.I + c->d.P, P = c->d.P;
    LCK(cudaMemcpyAsync(c->master + c->off_Wg, Wg_host, 4 * H * K * 4, cudaMemcpyHostToDevice, c->stream), "parameter upload");
    LCK(cudaMemcpyAsync(c->master + c->off_Wp, Wp_host, P * H * 4, cudaMemcpyHostToDevice, c->stream), "parameter upload");
    LCK(cudaMemcpyAsync(c->master + c->off_b, bias_host, 4 * H * 4, cudaMemcpyHostToDevice, c->stream), "parameter upload");
    // the FP16 working copies are the rounded masters (section 3.1); optimizer state restarts at zero
    LCK(launch_recast(c->master, c->w16, c->n_total, c->stream), "recast launch");
    if (c->s1) LCK(cudaMemsetAsync(c->s1, 0, c->n_total * 4, c->stream), "state clear");
    if (c->s2) LCK(cudaMemsetAsync(c->s2, 0, c->n_total * 4, c->stream), "state clear");
    LCK(cudaStreamSynchronize(c->stream), "stream synchronize");
    c->params_set = true;
    return MPT_OK;
}

int mpt_lstm_get_tensor(mpt_lstm_ctx *c, int kind, void *dst_host, size_t bytes)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!dst_host) return fail(c, MPT_ERR_INVALID_ARG, "null destination");
    const size_t T = c->d.T, B = c->d.B, I = c->d.I, H = c->d.H, P = c->d.P, K = I + P;
    const void *src = nullptr;
    size_t n = 0;
    switch (kind) {
        case MPT_LSTM_T_WG32: src = c->master + c->off_Wg; n = 4 * H * K * 4; break;
        case MPT_LSTM_T_WP32: src = c->master + c->off_Wp; n = P * H * 4; break;
        case MPT_LSTM_T_BIAS32: src = c->master + c->off_b; n = 4 * H * 4; break;
        case MPT_LSTM_T_WG16: src = c->w16 + c->off_Wg; n = 4 * H * K * 2; break;
        case MPT_LSTM_T_WP16: src = c->w16 + c->off_Wp; n = P * H * 2; break;
        case MPT_LSTM_T_BIAS16: src = c->w16 + c->off_b; n = 4 * H * 2; break;
        case MPT_LSTM_T_DWG16: src = c->g16 + c->off_Wg; n = 4 * H * K * 2; break;
        case MPT_LSTM_T_DWP16: src = c->g16 + c->off_Wp; n = P * H * 2; break;
        case MPT_LSTM_T_DBIAS16: src = c->g16 + c->off_b; n = 4 * H * 2; break;
        case MPT_LSTM_T_S1_WG32: if (!c->s1) return fail(c, MPT_ERR_STATE, "the optimizer keeps no first state"); src = c->s1 + c->off_Wg; n = 4 * H * K * 4; break;
        case MPT_LSTM_T_S1_WP32: if (!c->s1) return fail(c, MPT_ERR_STATE, "the optimizer keeps no first state"); src = c->s1 + c->off_Wp; n = P * H * 4; break;
        case MPT_LSTM_T_S1_BIAS32: if (!c->s1) return fail(c, MPT_ERR_STATE, "the optimizer keeps no first state"); src = c->s1 + c->off_b; n = 4 * H * 4; break;
        case MPT_LSTM_T_XR16: src = c->t.xr; n = (T + 1) * B * K * 2; break;
        case MPT_LSTM_T_DREXT16: src = c->t.dr_ext; n = T * B * P * 2; break;
        default: return fail(c, MPT_ERR_INVALID_ARG, "unknown tensor kind");
    }
    if (bytes != n) return fail(c, MPT_ERR_SHAPE, "byte count does not match the tensor");
    LCK(cudaMemcpyAsync(dst_host, src, n, cudaMemcpyDeviceToHost, c->stream), "tensor download");
    LCK(cudaStreamSynchronize(c->stream), "stream synchronize");
    return MPT_OK;
}

int mpt_lstm_set_dynamic_scale(mpt_lstm_ctx *c, int enable, int growth_interval, float min_scale, float max_scale)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (enable) {
        if (growth_interval < 1) return fail(c, MPT_ERR_INVALID_ARG, "growth interval must be >= 1");
        if (!valid_scale(min_scale) || !valid_scale(max_scale) || min_scale > max_scale)
            return fail(c, MPT_ERR_INVALID_ARG, "scale bounds out of range");
        uint32_t st[ST_WORDS];
        r = read_status(c, st, nullptr);
        if (r != MPT_OK) return r;
        memcpy(&c->S, &st[ST_SCALE], 4);
        c->growth_interval = growth_interval;
        c->scale_min = min_scale;
        c->scale_max = max_scale;
        c->S = fminf(fmaxf(c->S, min_scale), max_scale);
        c->dynamic_scale = true;
        return push_scale(c);
    }
    c->dynamic_scale = false;
    return MPT_OK;
}

int mpt_lstm_get_scale(mpt_lstm_ctx *c, float *S_out)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!S_out) return fail(c, MPT_ERR_INVALID_ARG, "null output");
    uint32_t st[ST_WORDS];
    r = read_status(c, st, nullptr);
    if (r != MPT_OK) return r;
    memcpy(S_out, &st[ST_SCALE], 4);
    c->S = *S_out;
    return MPT_OK;
}

int mpt_lstm_train_step(mpt_lstm_ctx *c, const uint16_t *x_dev, const int32_t *labels_dev, float *loss_host, int *overflow_host)
{
    int r = usable(c);
    if (r != MPT_OK) return r;
    if (!x_dev || !labels_dev) return fail(c, MPT_ERR_INVALID_ARG, "null input");
    if (!c->params_set) return fail(c, MPT_ERR_STATE, "mpt_lstm_train_step needs mpt_lstm_set_params first");
    const mpt_lstm_desc &d = c->d;
    const size_t T = d.T, B = d.B, I = d.I, H = d.H, P = d.P, K = I + P;
    cudaStream_t st = c->stream;
    // inputs into the left columns of the step rows; zero recurrent input and cell state at t = 0
    LCK(cudaMemcpy2DAsync(c->t.xr, K * 2, x_dev, I * 2, I * 2, T * B, cudaMemcpyDeviceToDevice, st), "input copy");
    LCK(cudaMemset2DAsync(c->t.xr + I, K * 2, 0, P * 2, B, st), "state clear");
    LCK(cudaMemsetAsync(c->t.c, 0, B * H * 2, st), "state clear");
    LCK(cudaMemsetAsync(c->status, 0, 3 * sizeof(uint32_t), st), "status clear");
    r = mpt_lstm_forward(&c->d, &c->t, st);
    if (r != MPT_OK) return fail(c, r, "LSTM forward failed to launch");
    // softmax cross-entropy on r_t as logits: rows (t, b) of the step rows' right-hand columns
    int nl = 0;
    cudaError_t e = launch_softmax_ce(c->t.xr + B * K + I, (int)K, labels_dev, (int)(T * B), (int)P, c->S, (uint16_t *)c->t.dr_ext,
                                      (int)P, c->row_loss, (float *)(c->status + ST_LOSS), c->status + ST_BAD_LABELS, st, &nl,
                                      (const float *)(c->status + ST_SCALE), c->status + ST_KERNEL_ERR);
    if (e != cudaSuccess) return cuda_fail(c, e, "softmax launch");
    r = mpt_lstm_backward(&c->d, &c->t, st);
    if (r != MPT_OK) return fail(c, r, "LSTM backward failed to launch");
    // master pass over the flat arena [Wg | Wp | bias] (padding holds zeros): unscale, skip on
    // overflow, optimizer step in FP32, re-round the FP16 copies
    LCK(cudaMemsetAsync(c->status + ST_OVERFLOW_SEEN, 0, sizeof(uint32_t), st), "status clear");
    const mpt_optimizer &o = c->opt;
    const float inv = 1.0f / c->S;
    if (o.clip_norm > 0.0f) {
        e = launch_clip_coef(c->g16, c->n_total, inv, (const float *)(c->status + ST_INV_SCALE), o.clip_norm, c->norm_parts,
                             (float *)(c->status + ST_CLIP_COEF), st);
        if (e != cudaSuccess) return cuda_fail(c, e, "clip launch");
    }
    if (o.kind == MPT_OPT_SGD && o.weight_decay == 0.0f && o.clip_norm <= 0.0f)
        e = launch_update(c->g16, c->master, c->s1, c->w16, c->n_total, inv, o.lr, o.momentum, c->s1 != nullptr,
                          c->status + ST_OVERFLOW, st, (const float *)(c->status + ST_INV_SCALE));
    else
        e = launch_update_opt(o.kind, c->g16, c->master, c->s1, c->s2, c->w16, c->n_total, inv, o.lr, o.momentum, o.beta2, o.eps,
                              o.weight_decay, 1.0f, 1.0f, c->status + ST_OVERFLOW, st, (const float *)(c->status + ST_INV_SCALE),
                              o.kind == MPT_OPT_ADAM ? (const float *)(c->status + ST_B1T) : nullptr,
                              o.clip_norm > 0.0f ? (const float *)(c->status + ST_CLIP_COEF) : nullptr);
    if (e != cudaSuccess) return cuda_fail(c, e, "update launch");
    if (c->dynamic_scale || o.kind == MPT_OPT_ADAM) {
        e = launch_post_step(c->status, c->dynamic_scale ? c->growth_interval : 0, 0.5f, 2.0f, c->scale_min, c->scale_max,
                             o.kind == MPT_OPT_ADAM ? 1 : 0, o.momentum, o.beta2, st);
        if (e != cudaSuccess) return cuda_fail(c, e, "post-step launch");
        }
    if (loss_host || overflow_host) {
        uint32_t w[ST_WORDS];
        r = read_status(c, w, nullptr);
        if (r != MPT_OK) return r;
        if (w[ST_OVERFLOW] == 0 && w[ST_OVERFLOW_SEEN] != 0)
            return fail(c, MPT_ERR_INTERNAL, "update kernel saw a non-finite gradient the producers did not flag");
        if (loss_host) memcpy(loss_host, &w[ST_LOSS], 4);
        if (overflow_host) *overflow_host = w[ST_OVERFLOW] ? 1 : 0;
        memcpy(&c->S, &w[ST_SCALE], 4);
        if (w[ST_BAD_LABELS] != 0) return fail(c, MPT_ERR_INVALID_ARG, "labels outside [0, P) were ignored");
    }
    return MPT_OK;
}

}  // extern "C"

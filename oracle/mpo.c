/*
 * mpo.c -- CPU oracle for the mixed-precision training hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * path computes, used by the test-suite and by the benchmark's CPU-baseline leg.
 * It shares no code with the CUDA library and the CUDA library never calls it.
 *
 * Recipe implemented (paper section 3; "pseudo FP16" mode of section 4):
 *   - tensors are stored as IEEE binary16 (section 3.1);
 *   - dot products multiply binary16 values and accumulate in binary32, the
 *     result is converted to binary16 when written (section 3.3);
 *   - reductions of the softmax are carried out in binary32 on binary16 data
 *     (section 3.3);
 *   - the loss is multiplied by a constant S before back-propagation, weight
 *     gradients are multiplied by 1/S before the update, an inf/NaN in the
 *     unscaled weight gradients skips the update (section 3.2);
 *   - the update is applied to a binary32 master copy which is then rounded to
 *     the binary16 working copy (section 3.1).
 *
 * The paper never names the rounding mode; round-to-nearest-even with gradual
 * underflow is used throughout.  The paper's sentence that magnitudes below
 * 2^-24 become zero (section 3.1) describes truncation; under round-to-nearest
 * values in (2^-25, 2^-24) round up to 2^-24 and 2^-25 itself ties to zero.
 *
 * Pins: every function here is checked by tests that do not go through this
 * file's own formulas (numpy's binary16 casts, exact rational arithmetic,
 * closed forms, finite differences in double precision).  No function is
 * "parity unpinned".
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 * (-ffp-contract=off keeps every binary32 operation separately rounded).
 * OpenMP is used over independent output rows / independent elements only, so
 * no element's arithmetic depends on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- binary16 */

static inline uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }
static inline float bits_f32(uint32_t u) { float x; memcpy(&x, &u, 4); return x; }

/* binary16 -> binary32, exact for every pattern (section 3.1: FP16 storage). */
float mpo_h2f(uint16_t h)
{
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1Fu;
    uint32_t m = h & 0x3FFu;
    if (e == 0x1Fu)                       /* inf / NaN */
        return bits_f32(sign | 0x7F800000u | (m << 13));
    if (e != 0)                           /* normal: exponent range [-14, 15] */
        return bits_f32(sign | ((e + 112u) << 23) | (m << 13));
    if (m == 0)
        return bits_f32(sign);
    /* subnormal: m * 2^-24 */
    float mag = (float)m * 0x1p-24f;
    return bits_f32(sign | f32_bits(mag));
}

/* binary32 -> binary16, round to nearest, ties to even, gradual underflow.
 * Largest finite result 65504; |x| >= 65520 becomes infinity (section 3.2). */
uint16_t mpo_f2h(float x)
{
    uint32_t u = f32_bits(x);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t a = u & 0x7FFFFFFFu;
    if (a > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);       /* NaN -> quiet NaN */
    if (a >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u);      /* >= 65520, inf */
    if (a >= 0x38800000u) {                                       /* >= 2^-14: normal */
        uint32_t e = (a >> 23) - 112u;
        uint32_t m = a & 0x7FFFFFu;
        uint32_t h = (e << 10) | (m >> 13);
        uint32_t rem = m & 0x1FFFu;
        if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) h++;   /* carry may bump the exponent */
        return (uint16_t)(sign | h);
    }
    /* result is subnormal or zero: round onto the 2^-24 grid */
    uint32_t e = a >> 23;
    if (e < 102u) return sign;                                    /* |x| < 2^-25 */
    uint32_t m = (a & 0x7FFFFFu) | 0x800000u;
    uint32_t shift = 126u - e;                                    /* 14 .. 24 */
    uint32_t h = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1u);
    if (rem > half || (rem == half && (h & 1u))) h++;
    return (uint16_t)(sign | h);
}

void mpo_h2f_array(const uint16_t *h, float *f, size_t n)
{
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; i++) f[i] = mpo_h2f(h[i]);
}

void mpo_f2h_array(const float *f, uint16_t *h, size_t n)
{
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; i++) h[i] = mpo_f2h(f[i]);
}

/* f2h over a contiguous range of binary32 bit patterns (exhaustive pin). */
void mpo_f2h_bits_range(uint32_t first, uint32_t count, uint16_t *h)
{
#pragma omp parallel for schedule(static)
    for (uint32_t i = 0; i < count; i++) h[i] = mpo_f2h(bits_f32(first + i));
}

int mpo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* -------------------------------------------------------------------- GEMM */
/*
 * C[m,n] = rn16( post( sum_{k ascending} A(m,k) * B(k,n) ) ), sum in binary32
 * (section 3.3: FP16 dot product accumulated in FP32, converted on the store).
 *
 * The three linear-layer products of one training iteration (section 3.1) differ
 * only in which index of each stored matrix is contracted:
 *   op 0 forward  Y = X W^T : A stored [M,K] (a_trans=0), B stored [N,K] (b_trans=0)
 *   op 1 dgrad    dX = dY W : A stored [M,K] (a_trans=0), B stored [K,N] (b_trans=1)
 *   op 2 wgrad    dW = dY^T X: A stored [K,M] (a_trans=1), B stored [K,N] (b_trans=1)
 * All stored matrices are row-major with leading dimensions lda/ldb/ldc.
 *
 * post: relu != 0 applies x>0 ? x : +0 to the binary32 sum before rounding
 *       (NaN propagates).  mask != NULL zeroes (+0) the rounded output where
 *       the stored binary16 value mask[m,n] is not > 0 (ReLU derivative taken
 *       from the stored activation).
 *
 * Side channels (optional, may be NULL): exact[m,n] = the same sum accumulated
 * in double (every product of two binary16 values is exact in double and the
 * double sum is accurate far below binary16 resolution); absdot[m,n] = sum |a*b|.
 *
 * row_begin/row_end restrict the computed output rows (used to time a slab).
 */
void mpo_gemm_f16(int op, int M, int N, int K,
                  const uint16_t *A, int lda, const uint16_t *B, int ldb,
                  uint16_t *C, int ldc, int relu,
                  const uint16_t *mask, int ldmask,
                  double *exact, double *absdot,
                  int row_begin, int row_end)
{
    const int a_trans = (op == 2);
    const int b_trans = (op != 0);
    if (row_begin < 0) row_begin = 0;
    if (row_end > M || row_end < 0) row_end = M;
    if (M <= 0 || N <= 0 || row_end <= row_begin) return;

    /* binary32 copy of the second operand laid out [K][N] so that, for a fixed
     * output row, the k loop is outermost and each output still sums k = 0..K-1
     * in ascending order. */
    float *Bf = (float *)malloc((size_t)(K > 0 ? K : 1) * (size_t)N * sizeof(float));
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++) {
            uint16_t hb = b_trans ? B[(size_t)k * ldb + n] : B[(size_t)n * ldb + k];
            Bf[(size_t)k * N + n] = mpo_h2f(hb);
        }

#pragma omp parallel
    {
        float *acc = (float *)malloc((size_t)N * sizeof(float));
        double *dacc = exact ? (double *)malloc((size_t)N * sizeof(double)) : NULL;
        double *aacc = absdot ? (double *)malloc((size_t)N * sizeof(double)) : NULL;
#pragma omp for schedule(static)
        for (int m = row_begin; m < row_end; m++) {
            for (int n = 0; n < N; n++) acc[n] = 0.0f;
            if (dacc) for (int n = 0; n < N; n++) dacc[n] = 0.0;
            if (aacc) for (int n = 0; n < N; n++) aacc[n] = 0.0;
            for (int k = 0; k < K; k++) {
                uint16_t ha = a_trans ? A[(size_t)k * lda + m] : A[(size_t)m * lda + k];
                float a = mpo_h2f(ha);
                const float *brow = Bf + (size_t)k * N;
                for (int n = 0; n < N; n++) {
                    float p = a * brow[n];          /* exact: <= 22 significant bits */
                    acc[n] = acc[n] + p;            /* one binary32 rounding per term */
                }
                if (dacc) for (int n = 0; n < N; n++) dacc[n] += (double)a * (double)brow[n];
                if (aacc) for (int n = 0; n < N; n++) aacc[n] += fabs((double)a * (double)brow[n]);
            }
            for (int n = 0; n < N; n++) {
                float s = acc[n];
                if (relu) s = (s > 0.0f) ? s : ((s != s) ? s : 0.0f);
                uint16_t h = mpo_f2h(s);
                if (mask && !(mpo_h2f(mask[(size_t)m * ldmask + n]) > 0.0f)) h = 0;
                C[(size_t)m * ldc + n] = h;
            }
            if (dacc) for (int n = 0; n < N; n++) exact[(size_t)m * N + n] = dacc[n];
            if (aacc) for (int n = 0; n < N; n++) absdot[(size_t)m * N + n] = aacc[n];
        }
        free(acc); free(dacc); free(aacc);
    }
    free(Bf);
}

/* One output element of the same product, for sampled checks at sizes where the
 * full product would take hours.  Returns the rounded binary16 (before mask). */
uint16_t mpo_gemm_f16_element(int op, int K,
                              const uint16_t *A, int lda, const uint16_t *B, int ldb,
                              int m, int n, int relu, double *exact, double *absdot)
{
    const int a_trans = (op == 2);
    const int b_trans = (op != 0);
    float acc = 0.0f;
    double d = 0.0, ad = 0.0;
    for (int k = 0; k < K; k++) {
        float a = mpo_h2f(a_trans ? A[(size_t)k * lda + m] : A[(size_t)m * lda + k]);
        float b = mpo_h2f(b_trans ? B[(size_t)k * ldb + n] : B[(size_t)n * ldb + k]);
        float p = a * b;
        acc = acc + p;
        d += (double)a * (double)b;
        ad += fabs((double)a * (double)b);
    }
    if (relu) acc = (acc > 0.0f) ? acc : ((acc != acc) ? acc : 0.0f);
    if (exact) *exact = d;
    if (absdot) *absdot = ad;
    return mpo_f2h(acc);
}

/* ------------------------------------------------ softmax cross-entropy */
/*
 * Per row i of binary16 logits z[i, 0..C-1] (section 3.3: reductions in FP32 on
 * FP16 data), with the loss scale S applied to the gradient (section 3.2: scaling
 * the loss scales every gradient by the chain rule):
 *   m = max_j z_j ; e_j = expf(z_j - m) ; s = sum_j e_j (ascending)
 *   loss_i = (m + logf(s)) - z_y
 *   c = S / (float)B ; dz[i,j] = rn16( (e_j / s - [j == y]) * c )
 * loss = (float)( sum_i (double)loss_i / B ), the unscaled mean.
 * A label outside [0, C) contributes no loss and a zero gradient row and is
 * counted in the return value.
 */
int mpo_softmax_ce(const uint16_t *z, int ldz, const int32_t *labels, int B, int C,
                   float S, uint16_t *dz, int lddz, float *row_loss, float *loss)
{
    int bad = 0;
    const float c = S / (float)B;
    float *rl = row_loss ? row_loss : (float *)malloc((size_t)(B > 0 ? B : 1) * sizeof(float));
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (int i = 0; i < B; i++) {
        const uint16_t *zi = z + (size_t)i * ldz;
        uint16_t *dzi = dz ? dz + (size_t)i * lddz : NULL;
        int y = labels[i];
        if (y < 0 || y >= C) {
            bad += 1;
            rl[i] = 0.0f;
            if (dzi) for (int j = 0; j < C; j++) dzi[j] = 0;
            continue;
        }
        float m = mpo_h2f(zi[0]);
        for (int j = 1; j < C; j++) {
            float v = mpo_h2f(zi[j]);
            if (v > m) m = v;                  /* a NaN logit reaches s through expf */
        }
        float s = 0.0f;
        for (int j = 0; j < C; j++) s = s + expf(mpo_h2f(zi[j]) - m);
        rl[i] = (m + logf(s)) - mpo_h2f(zi[y]);
        if (dzi)
            for (int j = 0; j < C; j++) {
                float e = expf(mpo_h2f(zi[j]) - m);
                float p = e / s;
                float d = p - ((j == y) ? 1.0f : 0.0f);
                dzi[j] = mpo_f2h(d * c);
            }
    }
    if (loss) {
        double acc = 0.0;
        for (int i = 0; i < B; i++) acc += (double)rl[i];
        *loss = (B > 0) ? (float)(acc / (double)B) : 0.0f;
    }
    if (!row_loss) free(rl);
    return bad;
}

/* ------------------------------------------------------- master-weight pass */
/*
 * Overflow inspection (section 3.2): 1 if any unscaled weight gradient
 * h2f(g[e]) * inv_S is inf or NaN.
 */
int mpo_grad_nonfinite(const uint16_t *g, size_t n, float inv_S)
{
    int flag = 0;
#pragma omp parallel for schedule(static) reduction(| : flag)
    for (size_t e = 0; e < n; e++) {
        float v = mpo_h2f(g[e]) * inv_S;
        if (!isfinite(v)) flag |= 1;
    }
    return flag;
}

/*
 * Update of the binary32 master copy and re-rounding of the binary16 working
 * copy (sections 3.1, 3.2).  Each line is one separately rounded binary32
 * operation (no fused multiply-add, no flush to zero):
 *   g = h2f(g16[e]) * inv_S
 *   momentum:  t = mu * v[e] ; v[e] = t + g ; u = lr * v[e]
 *   plain:     u = lr * g
 *   w32[e] = w32[e] - u ; w16[e] = rn16(w32[e])
 * The caller decides the skip: this function must only be called when
 * mpo_grad_nonfinite over ALL layers returned 0.
 */
void mpo_update_apply(const uint16_t *g16, float *w32, float *v, uint16_t *w16,
                      size_t n, float inv_S, float lr, float mu, int use_momentum)
{
#pragma omp parallel for schedule(static)
    for (size_t e = 0; e < n; e++) {
        float g = mpo_h2f(g16[e]) * inv_S;
        float u;
        if (use_momentum) {
            float t = mu * v[e];
            float nv = t + g;
            v[e] = nv;
            u = lr * nv;
        } else {
            u = lr * g;
        }
        float w = w32[e] - u;
        w32[e] = w;
        w16[e] = mpo_f2h(w);
    }
}

/*
 * Other optimizer steps on the binary32 master copy (the paper's experiments use Nesterov
 * momentum for the speech models, section 4.3; Adagrad for bigLSTM, section 4.5; Adam for
 * DCGAN, section 4.6; section 3.2 requires weight decay and other gradient-related terms to
 * act on the UNSCALED gradient).  The paper gives no formulas; the textbook forms are used,
 * every line one separately rounded binary32 operation, in this order:
 *   g = h2f(g16) * inv_S
 *   if wd != 0:          t = wd * w ; g = g + t                       (L2 weight decay)
 *   kind 1 Nesterov:     a = mu * s1 ; s1 = a + g ; b = mu * s1 ; c = g + b ; u = lr * c
 *   kind 2 Adagrad:      q = g * g ; s1 = s1 + q ; r = sqrtf(s1) ; d = r + eps ; c = g / d ; u = lr * c
 *   kind 3 Adam:         a = b1 * s1 ; b = omb1 * g ; s1 = a + b
 *                        q = g * g ; c = b2 * s2 ; d = omb2 * q ; s2 = c + d
 *                        mh = s1 / bc1 ; vh = s2 / bc2 ; r = sqrtf(vh) ; e = r + eps ; f = mh / e ; u = lr * f
 *     with omb1 = 1 - b1, omb2 = 1 - b2, bc1 = 1 - b1^t, bc2 = 1 - b2^t, where b1^t, b2^t are
 *     running binary32 products passed in by the caller (t counts applied, not skipped, steps)
 *   kind 0 SGD:          momentum (s1 != NULL): a = mu * s1 ; s1 = a + g ; u = lr * s1 ; else u = lr * g
 *   w = w - u ; w16 = rn16(w)
 * mu doubles as b1.  s1 / s2 may be NULL when the kind does not use them.
 */
/* One element of the steps listed above: g is the UNSCALED gradient; returns the new w. */
static inline float mpo_opt_elem(int kind, float g, float w, float *s1, float *s2, size_t i, float lr, float mu,
                                 float b2, float eps, float wd, float omb1, float omb2, float bc1, float bc2)
{
    if (wd != 0.0f) { float t = wd * w; g = g + t; }
    float u;
    if (kind == 1) {
        float a = mu * s1[i];
        float v = a + g;
        s1[i] = v;
        float b = mu * v;
        float c = g + b;
        u = lr * c;
    } else if (kind == 2) {
        float q = g * g;
        float h = s1[i] + q;
        s1[i] = h;
        float r = sqrtf(h);
        float d = r + eps;
        float c = g / d;
        u = lr * c;
    } else if (kind == 3) {
        float a = mu * s1[i];
        float b = omb1 * g;
        float m = a + b;
        s1[i] = m;
        float q = g * g;
        float c = b2 * s2[i];
        float d = omb2 * q;
        float v = c + d;
        s2[i] = v;
        float mh = m / bc1;
        float vh = v / bc2;
        float r = sqrtf(vh);
        float e = r + eps;
        float f = mh / e;
        u = lr * f;
    } else if (s1) {
        float a = mu * s1[i];
        float v = a + g;
        s1[i] = v;
        u = lr * v;
    } else {
        u = lr * g;
    }
    return w - u;
}

void mpo_update_apply_opt(int kind, const uint16_t *g16, float *w32, float *s1, float *s2, uint16_t *w16,
                          size_t n, float inv_S, float lr, float mu, float b2, float eps, float wd,
                          float bc1, float bc2)
{
    const float omb1 = 1.0f - mu, omb2 = 1.0f - b2;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; i++) {
        float g = mpo_h2f(g16[i]) * inv_S;
        float w = mpo_opt_elem(kind, g, w32[i], s1, s2, i, lr, mu, b2, eps, wd, omb1, omb2, bc1, bc2);
        w32[i] = w;
        w16[i] = mpo_f2h(w);
    }
}

/*
 * The same steps in the data-parallel setting of mpo_dp_update_apply (declared further down):
 * g = (h2f(g_0[i]) + h2f(g_1[i]) + ... in ascending replica order, binary32) * inv_SR, then the
 * lines above unchanged.  (Section 4.5: the language model trained over 4 GPUs uses Adagrad.)
 */
void mpo_dp_update_apply_opt(int kind, const uint16_t *const *g16, int R, float *w32, float *s1, float *s2,
                             uint16_t *w16, size_t n, float inv_SR, float lr, float mu, float b2, float eps,
                             float wd, float bc1, float bc2)
{
    const float omb1 = 1.0f - mu, omb2 = 1.0f - b2;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; i++) {
        float s = mpo_h2f(g16[0][i]);
        for (int q = 1; q < R; q++) s = s + mpo_h2f(g16[q][i]);
        float g = s * inv_SR;
        float w = mpo_opt_elem(kind, g, w32[i], s1, s2, i, lr, mu, b2, eps, wd, omb1, omb2, bc1, bc2);
        w32[i] = w;
        w16[i] = mpo_f2h(w);
    }
}

/*
 * Global-norm clipping in the data-parallel setting (section 3.2 puts clipping after unscaling;
 * section 4.5 aggregates the batch over several GPUs): the norm is that of the MEAN gradient the
 * update uses, g = (h2f(g_0[i]) + ... + h2f(g_{R-1}[i])) * inv_SR in binary32 as above, squares and
 * their sum in double; the update multiplies g by coef right after forming it, then the lines of
 * mpo_opt_elem unchanged.
 */
double mpo_dp_grad_sqnorm(const uint16_t *const *g16, int R, size_t n, float inv_SR)
{
    double total = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : total)
    for (size_t i = 0; i < n; i++) {
        float s = mpo_h2f(g16[0][i]);
        for (int q = 1; q < R; q++) s = s + mpo_h2f(g16[q][i]);
        float g = s * inv_SR;
        total += (double)g * (double)g;
    }
    return total;
}

void mpo_dp_update_apply_clip(int kind, const uint16_t *const *g16, int R, float *w32, float *s1, float *s2,
                              uint16_t *w16, size_t n, float inv_SR, float coef, float lr, float mu, float b2,
                              float eps, float wd, float bc1, float bc2)
{
    const float omb1 = 1.0f - mu, omb2 = 1.0f - b2;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; i++) {
        float s = mpo_h2f(g16[0][i]);
        for (int q = 1; q < R; q++) s = s + mpo_h2f(g16[q][i]);
        float g = s * inv_SR;
        g = g * coef;
        float w = mpo_opt_elem(kind, g, w32[i], s1, s2, i, lr, mu, b2, eps, wd, omb1, omb2, bc1, bc2);
        w32[i] = w;
        w16[i] = mpo_f2h(w);
    }
}

/*
 * Sum of squares of the unscaled weight gradients, accumulated in double (section 3.2: gradient
 * clipping acts on the unscaled gradients; section 3.3: reductions are carried out in higher
 * precision than the stored values).  Global-norm clipping then multiplies every unscaled
 * gradient by coef = min(1, clip / (sqrt(total) + 1e-6)) rounded to binary32.
 */
double mpo_grad_sqnorm(const uint16_t *g, size_t n, float inv_S)
{
    double total = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : total)
    for (size_t e = 0; e < n; e++) {
        float v = mpo_h2f(g[e]) * inv_S;
        total += (double)v * (double)v;
    }
    return total;
}

/* mpo_update_apply_opt with the clipping coefficient applied right after unscaling:
 *   g = h2f(g16) * inv_S ; g = g * coef ; then weight decay and the optimizer step as above. */
void mpo_update_apply_clip(int kind, const uint16_t *g16, float *w32, float *s1, float *s2, uint16_t *w16,
                           size_t n, float inv_S, float coef, float lr, float mu, float b2, float eps, float wd,
                           float bc1, float bc2)
{
    const float omb1 = 1.0f - mu, omb2 = 1.0f - b2;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; i++) {
        float g = mpo_h2f(g16[i]) * inv_S;
        g = g * coef;
        float w = mpo_opt_elem(kind, g, w32[i], s1, s2, i, lr, mu, b2, eps, wd, omb1, omb2, bc1, bc2);
        w32[i] = w;
        w16[i] = mpo_f2h(w);
    }
}

/* ------------------------------------------------------------------------
 * LSTM cell with fused gate arithmetic (sections 3.3 and 4.5: recurrent matrix products on
 * FP16 inputs with FP32 accumulation; point-wise gate arithmetic is memory-bound and may run
 * in either precision - here FP32 arithmetic on FP16 storage).
 *
 * Row b of XR holds [x_t ; r_{t-1}] (K values).  Wg is [4H][K], row 4j+q = gate q of cell j
 * with q: 0 input, 1 forget, 2 candidate, 3 output; bias16 [4H] in the same order.
 *   pre_q = (sum_k XR[b,k]*Wg[4j+q,k], ascending k, binary32) + h2f(bias16[4j+q])
 *   i = sig(pre_0)  f = sig(pre_1)  g = tanh(pre_2)  o = sig(pre_3),  sig(x) = 1/(1+exp(-x))
 *   acts[b,4j+q] = rn16(gate value)
 *   c = f*c_prev + i*g  (two products, one sum, each rounded to binary32);  c16 = rn16(c)
 *   h16 = rn16(o * tanh(h2f(c16)))     (consumers only ever see the stored cell state)
 * pre32 (optional) receives the binary32 pre-activations, absdot (optional) sum |a*b| per gate.
 */
static float mpo_sigmoid(float x)
{
    float e = expf(-x);
    float d = 1.0f + e;
    return 1.0f / d;
}

void mpo_lstm_cell_fwd(int B, int H, int K, const uint16_t *XR, int ldxr, const uint16_t *Wg, int ldw,
                       const uint16_t *bias16, const uint16_t *c_prev, int ldcp, uint16_t *acts, int ldacts,
                       uint16_t *c_out, int ldco, uint16_t *h_out, int ldh, float *pre32, double *absdot)
{
    const int N = 4 * H;
    float *Wf = (float *)malloc((size_t)(K > 0 ? K : 1) * (size_t)N * sizeof(float));   /* [K][N] */
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++) Wf[(size_t)k * N + n] = mpo_h2f(Wg[(size_t)n * ldw + k]);
#pragma omp parallel
    {
        float *acc = (float *)malloc((size_t)N * sizeof(float));
        double *aacc = (double *)malloc((size_t)N * sizeof(double));
#pragma omp for schedule(static)
        for (int b = 0; b < B; b++) {
            for (int n = 0; n < N; n++) { acc[n] = 0.0f; aacc[n] = 0.0; }
            for (int k = 0; k < K; k++) {
                float a = mpo_h2f(XR[(size_t)b * ldxr + k]);
                const float *wrow = Wf + (size_t)k * N;
                for (int n = 0; n < N; n++) {
                    float p = a * wrow[n];
                    acc[n] = acc[n] + p;
                    aacc[n] += fabs((double)a * (double)wrow[n]);
                }
            }
            for (int j = 0; j < H; j++) {
                float pre[4];
                for (int q = 0; q < 4; q++) {
                    pre[q] = acc[4 * j + q] + mpo_h2f(bias16[4 * j + q]);
                    if (pre32) pre32[(size_t)b * N + 4 * j + q] = pre[q];
                    if (absdot) absdot[(size_t)b * N + 4 * j + q] = aacc[4 * j + q];
                }
                float gi = mpo_sigmoid(pre[0]), gf = mpo_sigmoid(pre[1]), gg = tanhf(pre[2]), go = mpo_sigmoid(pre[3]);
                uint16_t *arow = acts + (size_t)b * ldacts + 4 * j;
                arow[0] = mpo_f2h(gi); arow[1] = mpo_f2h(gf); arow[2] = mpo_f2h(gg); arow[3] = mpo_f2h(go);
                float cp = mpo_h2f(c_prev[(size_t)b * ldcp + j]);
                float t1 = gf * cp;
                float t2 = gi * gg;
                float c = t1 + t2;
                uint16_t c16 = mpo_f2h(c);
                c_out[(size_t)b * ldco + j] = c16;
                float tc = tanhf(mpo_h2f(c16));
                float h = go * tc;
                h_out[(size_t)b * ldh + j] = mpo_f2h(h);
            }
        }
        free(acc);
        free(aacc);
    }
    free(Wf);
}

/*
 * Backward of the gate arithmetic for one time step, from stored FP16 values (the chain rule
 * of the forward formulas; every operation one binary32 rounding, in the order written):
 *   tc = tanh(h2f(c16));  dh, dc_next: scaled gradients wrt h_t and (from step t+1) wrt c_t
 *   dc  = (dh*o)*(1 - tc*tc) + dc_next
 *   dpre_o = (dh*tc) * (o*(1-o))
 *   dpre_i = (dc*g)  * (i*(1-i))
 *   dpre_f = (dc*cp) * (f*(1-f))
 *   dpre_g = (dc*i)  * (1 - g*g)
 *   dc_prev = dc*f
 * dG[b,4j+q] = rn16(dpre_q), dc_prev16 = rn16(dc_prev).  dc_next may be NULL (last step: zero).
 */
void mpo_lstm_cell_bwd(int B, int H, const uint16_t *dh, int lddh, const uint16_t *dc_next, int lddc,
                       const uint16_t *acts, int ldacts, const uint16_t *c_prev, int ldcp, const uint16_t *c16,
                       int ldc, uint16_t *dG, int lddg, uint16_t *dc_prev, int lddcp)
{
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; b++)
        for (int j = 0; j < H; j++) {
            const uint16_t *arow = acts + (size_t)b * ldacts + 4 * j;
            float gi = mpo_h2f(arow[0]), gf = mpo_h2f(arow[1]), gg = mpo_h2f(arow[2]), go = mpo_h2f(arow[3]);
            float cp = mpo_h2f(c_prev[(size_t)b * ldcp + j]);
            float tc = tanhf(mpo_h2f(c16[(size_t)b * ldc + j]));
            float dhv = mpo_h2f(dh[(size_t)b * lddh + j]);
            float dcn = dc_next ? mpo_h2f(dc_next[(size_t)b * lddc + j]) : 0.0f;
            float a1 = dhv * go;
            float a2 = tc * tc;
            float a3 = 1.0f - a2;
            float a4 = a1 * a3;
            float dc = a4 + dcn;
            float o1 = dhv * tc;
            float o2 = 1.0f - go;
            float o3 = go * o2;
            float dpo = o1 * o3;
            float i1 = dc * gg;
            float i2 = 1.0f - gi;
            float i3 = gi * i2;
            float dpi = i1 * i3;
            float f1 = dc * cp;
            float f2 = 1.0f - gf;
            float f3 = gf * f2;
            float dpf = f1 * f3;
            float g1 = dc * gi;
            float g2 = gg * gg;
            float g3 = 1.0f - g2;
            float dpg = g1 * g3;
            float dcp = dc * gf;
            uint16_t *drow = dG + (size_t)b * lddg + 4 * j;
            drow[0] = mpo_f2h(dpi); drow[1] = mpo_f2h(dpf); drow[2] = mpo_f2h(dpg); drow[3] = mpo_f2h(dpo);
            dc_prev[(size_t)b * lddcp + j] = mpo_f2h(dcp);
        }
}

/* Bias gradient: column sums of the FP16 gate gradients over all rows, accumulated in binary32
 * in ascending row order (section 3.3: reductions in FP32), rounded to FP16 on store. */
void mpo_bias_grad(const uint16_t *dG, size_t rows, int cols, int ld, uint16_t *db16, float *db32)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < cols; n++) {
        float s = 0.0f;
        for (size_t r = 0; r < rows; r++) s = s + mpo_h2f(dG[r * (size_t)ld + n]);
        if (db32) db32[n] = s;
        db16[n] = mpo_f2h(s);
    }
}

/* out = rn16(h2f(a) + h2f(b)) element-wise over a [rows, cols] block (gradient of a value that is
 * consumed twice: by the layer above and by the next time step). */
void mpo_add_f16(const uint16_t *a, int lda, const uint16_t *b, int ldb, uint16_t *out, int ldo, int rows, int cols)
{
    for (int r = 0; r < rows; r++)
        for (int n = 0; n < cols; n++) {
            float s = mpo_h2f(a[(size_t)r * lda + n]) + mpo_h2f(b[(size_t)r * ldb + n]);
            out[(size_t)r * ldo + n] = mpo_f2h(s);
        }
}

/*
 * One data-parallel step over R replicas of the model (section 4.5 trains with a batch aggregated
 * over 4 GPUs; the paper gives no formulas for the exchange, so the plain definition is used: the
 * gradient of the mean loss over the aggregated batch is the mean of the replicas' gradients).
 * Every replica holds a loss-scaled binary16 gradient g_q; per element, each line one separately
 * rounded binary32 operation:
 *   s = h2f(g_0[e]) ; for q = 1 .. R-1 in ascending order: s = s + h2f(g_q[e])
 *   g = s * inv_SR                    inv_SR = 1 / (S * R), formed by the caller in binary32
 *   then the momentum / plain lines of mpo_update_apply:  v, w32, w16 = rn16(w32)
 * The sum stays in binary32 (it is never stored as binary16), so it cannot overflow when its
 * terms are finite.  The caller decides the skip: this function must only be called when
 * mpo_grad_nonfinite returned 0 for EVERY replica's gradient.
 */
void mpo_dp_update_apply(const uint16_t *const *g16, int R, float *w32, float *v, uint16_t *w16,
                         size_t n, float inv_SR, float lr, float mu, int use_momentum)
{
#pragma omp parallel for schedule(static)
    for (size_t e = 0; e < n; e++) {
        float s = mpo_h2f(g16[0][e]);
        for (int q = 1; q < R; q++) s = s + mpo_h2f(g16[q][e]);
        float g = s * inv_SR;
        float u;
        if (use_momentum) {
            float t = mu * v[e];
            float nv = t + g;
            v[e] = nv;
            u = lr * nv;
        } else {
            u = lr * g;
        }
        float w = w32[e] - u;
        w32[e] = w;
        w16[e] = mpo_f2h(w);
    }
}

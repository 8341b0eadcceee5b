/*
 * CPU oracle, C twin: the delayed synchronous step of ABS-SGD (arXiv 2308.15164,
 * Algorithm 1), written as plain loops.
 *
 * TEST INFRASTRUCTURE ONLY.  It shares no code with the CUDA path.  Tests compare it with
 * the NumPy oracle (two independent plain implementations) and the benchmark times it on
 * the host cores as the reported CPU baseline.  OpenMP only splits the element loops; no
 * blocking, fusion or reordering beyond Algorithm 1's own steps.
 *
 * State and update rule are those of oracle/abs_oracle.py:
 *   accumulate(i, g):  G_t^i += g (fp32, call order);  b_i += 1          (Algorithm 1, Step 2)
 *   sync_step():       d = cur^1;  B = sum_i b_i[d]
 *                      if B > 0:  Gbar = (sum_i G^i[d]) / B               (Algorithm 1, Step 1)
 *                                 Gbar += lambda * Gbar*Gbar*(x - x_prev)  (Eq. 6)
 *                                 g = Gbar + wd*x;  v = mu*v + g;  x -= lr*v
 *                      x_prev = old x;  G[d] = 0;  b[d] = 0;  cur = d;  t += 1
 * x, v are held in fp64 and rounded to fp32 only on output.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    size_t P;
    int W;
    double lr, mu, wd, lambda_dc;
    double *x, *x_prev, *v;
    float *acc;      /* [2][W][P] */
    int64_t *cnt;    /* [2][W]    */
    int cur;
    int64_t t;
} abs_oracle;

abs_oracle *abs_oracle_create(size_t P, int W, const float *x0, double lr, double mu, double wd,
                              double lambda_dc) {
    abs_oracle *o = (abs_oracle *)calloc(1, sizeof(abs_oracle));
    if (!o) return NULL;
    o->P = P; o->W = W; o->lr = lr; o->mu = mu; o->wd = wd; o->lambda_dc = lambda_dc;
    o->x = (double *)malloc(P * sizeof(double));
    o->x_prev = (double *)malloc(P * sizeof(double));
    o->v = (double *)calloc(P, sizeof(double));
    o->acc = (float *)calloc((size_t)2 * W * P, sizeof(float));
    o->cnt = (int64_t *)calloc((size_t)2 * W, sizeof(int64_t));
    if (!o->x || !o->x_prev || !o->v || !o->acc || !o->cnt) return NULL;
    for (size_t j = 0; j < P; ++j) { o->x[j] = (double)x0[j]; o->x_prev[j] = o->x[j]; }
    return o;
}

void abs_oracle_destroy(abs_oracle *o) {
    if (!o) return;
    free(o->x); free(o->x_prev); free(o->v); free(o->acc); free(o->cnt); free(o);
}

static float bf16_widen(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* dtype 0: g points at fp32 values; dtype 1: g points at bf16 bit patterns. */
int abs_oracle_accumulate(abs_oracle *o, int i, const void *g, int dtype) {
    if (i < 0 || i >= o->W) return -1;
    float *row = o->acc + ((size_t)o->cur * o->W + i) * o->P;
    const size_t P = o->P;
    if (dtype == 0) {
        const float *gf = (const float *)g;
#pragma omp parallel for schedule(static)
        for (size_t j = 0; j < P; ++j) row[j] += gf[j];
    } else {
        const uint16_t *gb = (const uint16_t *)g;
#pragma omp parallel for schedule(static)
        for (size_t j = 0; j < P; ++j) row[j] += bf16_widen(gb[j]);
    }
    o->cnt[o->cur * o->W + i] += 1;
    return 0;
}

/* Returns B, the total micro-batch count the step consumed; writes the W consumed b_i to b_out. */
int64_t abs_oracle_sync_step(abs_oracle *o, int32_t *b_out) {
    const int d = o->cur ^ 1;
    const size_t P = o->P;
    const int W = o->W;
    int64_t B = 0;
    for (int i = 0; i < W; ++i) {
        B += o->cnt[d * W + i];
        if (b_out) b_out[i] = (int32_t)o->cnt[d * W + i];
    }
    float *set = o->acc + (size_t)d * W * P;
    const double lr = o->lr, mu = o->mu, wd = o->wd, lam = o->lambda_dc;
#pragma omp parallel for schedule(static)
    for (size_t j = 0; j < P; ++j) {
        const double x_old = o->x[j];
        if (B > 0) {
            double G = 0.0;
            for (int i = 0; i < W; ++i) G += (double)set[(size_t)i * P + j];
            double Gbar = G / (double)B;
            if (lam != 0.0) Gbar = Gbar + lam * Gbar * Gbar * (x_old - o->x_prev[j]);
            const double g = Gbar + wd * x_old;
            const double vn = mu * o->v[j] + g;
            o->v[j] = vn;
            o->x[j] = x_old - lr * vn;
        }
        o->x_prev[j] = x_old;
        for (int i = 0; i < W; ++i) set[(size_t)i * P + j] = 0.0f;
    }
    for (int i = 0; i < W; ++i) o->cnt[d * W + i] = 0;
    o->cur = d;
    o->t += 1;
    return B;
}

void abs_oracle_params(const abs_oracle *o, float *out) {
    for (size_t j = 0; j < o->P; ++j) out[j] = (float)o->x[j];
}

void abs_oracle_momentum(const abs_oracle *o, double *out) {
    memcpy(out, o->v, o->P * sizeof(double));
}

void abs_oracle_state(const abs_oracle *o, int32_t *cnt_out /* [2][W] */, int32_t *cur, int64_t *t) {
    for (int k = 0; k < 2 * o->W; ++k) cnt_out[k] = (int32_t)o->cnt[k];
    *cur = o->cur;
    *t = o->t;
}

void abs_oracle_set_lr(abs_oracle *o, double lr) { o->lr = lr; }

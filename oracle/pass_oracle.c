/*
 * CPU oracle of the PaSS decoder forward: TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, float64 implementation of one multi-token forward pass of a
 * LLaMA-style decoder with a KV cache ("a single forward pass on n tokens in
 * parallel", Method / Speculative Sampling; "re-implementation of the 7B LLaMa
 * model", Experiments).  It shares no code with the CUDA library and is only
 * called from tests, the smoke check and the CPU-baseline leg of the benchmark.
 *
 * Weights are read at their exact stored values (float32, or bfloat16 widened
 * bit-exactly); every activation, the KV cache and every accumulator is double.
 * Each output row is accumulated over k = 0, 1, 2, ... in that order, whatever
 * other rows share the call, so a row's result does not depend on its
 * neighbours: n rows in one call equal n calls of one row bit for bit.
 * Compile with -ffp-contract=off so that vectorised and scalar loops round alike.
 *
 * Architecture reading (the paper only says "7B LLaMa"): pre-norm residual
 * blocks, RMSNorm, rotary positions on adjacent pairs (2i, 2i+1) with angle
 * pos * theta^(-2i/d_head), multi-head attention with n_kv = n_heads, SwiGLU
 * feed-forward, no biases, untied output head.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int n_layers, d_model, n_heads, d_head, d_ffn, vocab;
    int wdtype;                 /* 0 = float32, 1 = bfloat16 (uint16 bit patterns) */
    int kvdtype;                /* how a K/V row is stored: 0 = as computed (float64), 1 = rounded to bfloat16 */
    double rms_eps, rope_theta;
    const void *lm_head, *final_norm;
    const void *const *wq, *const *wk, *const *wv, *const *wo;
    const void *const *wg, *const *wu, *const *wd;
    const void *const *norm_attn, *const *norm_ffn;
} oracle_model;

static inline double w_at(const void *w, int dtype, size_t i) {
    if (dtype == 0) return (double)((const float *)w)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)w)[i]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

/* Nearest bfloat16 (sign, 8 exponent bits, 7 fraction bits), ties to even, of a double in bfloat16's
 * normal range; zero, and anything outside that range, is returned as it is. */
static inline double to_bf16(double x) {
    const double ax = fabs(x);
    if (!(ax >= 0x1p-126 && ax < 0x1p127)) return x;
    uint64_t b;
    memcpy(&b, &x, 8);
    const uint64_t drop = 52 - 7;                      /* fraction bits that do not fit */
    b += (((uint64_t)1 << (drop - 1)) - 1) + ((b >> drop) & 1);
    b &= ~(((uint64_t)1 << drop) - 1);
    memcpy(&x, &b, 8);
    return x;
}

/* y[r][o] = sum_k x[r][k] * W[o][k]   (W is [n_out][n_in] row-major) */
static void linear(const oracle_model *m, const void *W, int n_out, int n_in,
                   const double *x, int n_rows, double *y) {
    /* xT[k][r] so that the inner loop runs over rows with one weight value */
    double *xT = (double *)malloc(sizeof(double) * (size_t)n_in * n_rows);
    for (int r = 0; r < n_rows; r++)
        for (int k = 0; k < n_in; k++) xT[(size_t)k * n_rows + r] = x[(size_t)r * n_in + k];
#pragma omp parallel
    {
        double *acc = (double *)malloc(sizeof(double) * n_rows);
#pragma omp for schedule(static)
        for (int o = 0; o < n_out; o++) {
            for (int r = 0; r < n_rows; r++) acc[r] = 0.0;
            for (int k = 0; k < n_in; k++) {
                const double wk = w_at(W, m->wdtype, (size_t)o * n_in + k);
                const double *xk = xT + (size_t)k * n_rows;
                for (int r = 0; r < n_rows; r++) acc[r] += xk[r] * wk;
            }
            for (int r = 0; r < n_rows; r++) y[(size_t)r * n_out + o] = acc[r];
        }
        free(acc);
    }
    free(xT);
}

/* y = x * g / sqrt(mean(x^2) + eps), row by row */
static void rmsnorm(const oracle_model *m, const void *g, const double *x, int n_rows, double *y) {
    const int d = m->d_model;
    for (int r = 0; r < n_rows; r++) {
        double ss = 0.0;
        for (int i = 0; i < d; i++) ss += x[(size_t)r * d + i] * x[(size_t)r * d + i];
        const double inv = 1.0 / sqrt(ss / d + m->rms_eps);
        for (int i = 0; i < d; i++)
            y[(size_t)r * d + i] = x[(size_t)r * d + i] * inv * w_at(g, m->wdtype, i);
    }
}

/* rotate pairs (2i, 2i+1) of every head by pos * theta^(-2i/d_head) */
static void rope(const oracle_model *m, double *v, int pos) {
    const int dh = m->d_head;
    for (int h = 0; h < m->n_heads; h++)
        for (int i = 0; i < dh / 2; i++) {
            const double ang = (double)pos * pow(m->rope_theta, -2.0 * i / dh);
            const double c = cos(ang), s = sin(ang);
            double *p = v + (size_t)h * dh + 2 * i;
            const double a = p[0], b = p[1];
            p[0] = a * c - b * s;
            p[1] = a * s + b * c;
        }
}

/*
 * Causal softmax attention of n_rows queries against one layer's cache.
 * q, o: [n_rows][d_model]; kc, vc: [>= pos0+n_rows][d_model].  Row r, head h:
 * o = sum_{j <= pos0+r} softmax_j(q.k_j / sqrt(d_head)) v_j.
 */
static void attention(const oracle_model *m, const double *q, const double *kc, const double *vc,
                      int n_rows, int pos0, double *o) {
    const int d = m->d_model, H = m->n_heads, dh = m->d_head;
    const double scale = 1.0 / sqrt((double)dh);
#pragma omp parallel for collapse(2) schedule(static)
    for (int r = 0; r < n_rows; r++)
        for (int hd = 0; hd < H; hd++) {
            const int n_keys = pos0 + r + 1;
            double *s = (double *)malloc(sizeof(double) * n_keys);
            const double *qh = q + (size_t)r * d + (size_t)hd * dh;
            double mx = -INFINITY;
            for (int j = 0; j < n_keys; j++) {
                const double *kj = kc + (size_t)j * d + (size_t)hd * dh;
                double dot = 0.0;
                for (int i = 0; i < dh; i++) dot += qh[i] * kj[i];
                s[j] = dot * scale;
                if (s[j] > mx) mx = s[j];
            }
            double den = 0.0;
            for (int j = 0; j < n_keys; j++) { s[j] = exp(s[j] - mx); den += s[j]; }
            double *oh = o + (size_t)r * d + (size_t)hd * dh;
            for (int i = 0; i < dh; i++) oh[i] = 0.0;
            for (int j = 0; j < n_keys; j++) {
                const double p = s[j] / den;
                const double *vj = vc + (size_t)j * d + (size_t)hd * dh;
                for (int i = 0; i < dh; i++) oh[i] += p * vj[i];
            }
            free(s);
        }
}

/* SwiGLU gate: silu(g) * u with silu(x) = x / (1 + exp(-x)) */
static void swiglu(double *g, const double *u, size_t n) {
    for (size_t i = 0; i < n; i++) g[i] = g[i] / (1.0 + exp(-g[i])) * u[i];
}

/*
 * Forward of n_rows input vectors x_in[r] (token or look-ahead embeddings, already
 * gathered, double) placed at positions pos0 .. pos0+n_rows-1 of one sequence.
 * kcache / vcache: [n_layers][kv_capacity][d_model] doubles; rows pos0.. are written,
 * rows 0..pos0-1 are read.  Row r attends to positions 0 .. pos0+r (causal).
 * logits_out: [n_rows][vocab], or NULL to skip the output head (prompt processing).
 * hidden_out: optional [n_rows][d_model] final residual stream (before the last norm).
 * Returns 0, or -1 on a bad argument.
 */
int oracle_forward(const oracle_model *m, const double *x_in, int n_rows, int pos0,
                   double *kcache, double *vcache, int kv_capacity,
                   double *logits_out, double *hidden_out) {
    if (!m || !x_in || n_rows <= 0 || pos0 < 0 || pos0 + n_rows > kv_capacity) return -1;
    const int d = m->d_model, f = m->d_ffn, H = m->n_heads, dh = m->d_head;
    if (H * dh != d) return -1;
    const size_t nd = (size_t)n_rows * d;
    double *h = (double *)malloc(sizeof(double) * nd);
    double *a = (double *)malloc(sizeof(double) * nd);
    double *q = (double *)malloc(sizeof(double) * nd);
    double *kk = (double *)malloc(sizeof(double) * nd);
    double *vv = (double *)malloc(sizeof(double) * nd);
    double *o = (double *)malloc(sizeof(double) * nd);
    double *t = (double *)malloc(sizeof(double) * nd);
    double *g = (double *)malloc(sizeof(double) * (size_t)n_rows * f);
    double *u = (double *)malloc(sizeof(double) * (size_t)n_rows * f);
    memcpy(h, x_in, sizeof(double) * nd);

    for (int l = 0; l < m->n_layers; l++) {
        double *kc = kcache + (size_t)l * kv_capacity * d;
        double *vc = vcache + (size_t)l * kv_capacity * d;
        /* attention block */
        rmsnorm(m, m->norm_attn[l], h, n_rows, a);
        linear(m, m->wq[l], d, d, a, n_rows, q);
        linear(m, m->wk[l], d, d, a, n_rows, kk);
        linear(m, m->wv[l], d, d, a, n_rows, vv);
        for (int r = 0; r < n_rows; r++) {
            rope(m, q + (size_t)r * d, pos0 + r);
            rope(m, kk + (size_t)r * d, pos0 + r);
            /* the cache holds what its storage format can hold; attention reads the cache */
            for (int i = 0; i < d; i++) {
                const double kx = kk[(size_t)r * d + i], vx = vv[(size_t)r * d + i];
                kc[(size_t)(pos0 + r) * d + i] = m->kvdtype == 1 ? to_bf16(kx) : kx;
                vc[(size_t)(pos0 + r) * d + i] = m->kvdtype == 1 ? to_bf16(vx) : vx;
            }
        }
        attention(m, q, kc, vc, n_rows, pos0, o);
        linear(m, m->wo[l], d, d, o, n_rows, t);
        for (size_t i = 0; i < nd; i++) h[i] += t[i];
        /* feed-forward block: h += (silu(b Wg^T) * (b Wu^T)) Wd^T */
        rmsnorm(m, m->norm_ffn[l], h, n_rows, a);
        linear(m, m->wg[l], f, d, a, n_rows, g);
        linear(m, m->wu[l], f, d, a, n_rows, u);
        swiglu(g, u, (size_t)n_rows * f);
        linear(m, m->wd[l], d, f, g, n_rows, t);
        for (size_t i = 0; i < nd; i++) h[i] += t[i];
    }
    if (hidden_out) memcpy(hidden_out, h, sizeof(double) * nd);
    if (logits_out) {
        rmsnorm(m, m->final_norm, h, n_rows, a);
        linear(m, m->lm_head, m->vocab, d, a, n_rows, logits_out);
    }
    free(h); free(a); free(q); free(kk); free(vv); free(o); free(t); free(g); free(u);
    return 0;
}

/* Single pieces, exported so that tests can pin them one by one. */
int oracle_linear(const oracle_model *m, const void *W, int n_out, int n_in,
                  const double *x, int n_rows, double *y) {
    linear(m, W, n_out, n_in, x, n_rows, y);
    return 0;
}

int oracle_rmsnorm(const oracle_model *m, const void *g, const double *x, int n_rows, double *y) {
    rmsnorm(m, g, x, n_rows, y);
    return 0;
}

int oracle_rope(const oracle_model *m, double *v, int pos) {
    rope(m, v, pos);
    return 0;
}

int oracle_attention(const oracle_model *m, const double *q, const double *kc, const double *vc,
                     int n_rows, int pos0, double *o) {
    attention(m, q, kc, vc, n_rows, pos0, o);
    return 0;
}

int oracle_swiglu(double *g, const double *u, long n) {
    swiglu(g, u, (size_t)n);
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

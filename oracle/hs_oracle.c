/* CPU oracle - see hs_oracle.h.  TEST INFRASTRUCTURE ONLY. */
#include "hs_oracle.h"
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ helpers */
static inline double bf16_val(uint16_t b) {
    uint32_t u = (uint32_t)b << 16; float f; memcpy(&f, &u, 4); return (double)f;
}
static inline uint16_t to_bf16(double x) {   /* double -> float32 -> bf16, round to nearest even */
    float f = (float)x; uint32_t u; memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
static inline double silu(double x) { return x / (1.0 + exp(-x)); }
static inline double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }
static inline double softplus(double x) { return x > 30.0 ? x : log1p(exp(x)); }

/* --------------------------------------------------------------- components */
/* RMSNorm: out_i = x_i / sqrt(mean(x^2) + eps) * w_i */
void or_rmsnorm(const double *x, const float *w, int n, double eps, double *out) {
    double ss = 0.0;
    for (int i = 0; i < n; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / n + eps);
    for (int i = 0; i < n; ++i) out[i] = x[i] * r * (double)w[i];
}

/* y = W x, W bf16 [rows, cols] row-major with a row stride */
void or_matvec(const uint8_t *blob, or_mat W, int rows, int cols, const double *x, double *y) {
    const uint16_t *w0 = (const uint16_t *)(blob + W.off);
#pragma omp parallel for schedule(static) if ((int64_t)rows * cols > 65536)
    for (int r = 0; r < rows; ++r) {
        const uint16_t *w = w0 + (int64_t)r * W.stride;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int j = 0; j < cols; ++j) acc += bf16_val(w[j]) * x[j];
        y[r] = acc;
    }
}

/* causal depthwise conv, one channel, one new input: taps[3] multiplies the newest input */
double or_conv_step(double *win3, double cur, const float *taps4, double bias) {
    double o = bias + taps4[0] * win3[0] + taps4[1] * win3[1] + taps4[2] * win3[2] + taps4[3] * cur;
    win3[0] = win3[1]; win3[1] = win3[2]; win3[2] = cur;
    return o;
}

/* Mamba-2 recurrence for one head: S <- exp(dt A) S + dt x (x) B ; y = S C + D x */
void or_ssm_step(double *S, int P, int N, double dt, double A, double Dh,
                 const double *x, const double *B, const double *C, double *y) {
    double a = exp(dt * A);
    for (int p = 0; p < P; ++p) {
        double acc = 0.0;
        for (int n = 0; n < N; ++n) {
            double s = a * S[p * N + n] + dt * x[p] * B[n];
            S[p * N + n] = s;
            acc += s * C[n];
        }
        y[p] = acc + Dh * x[p];
    }
}

/* The same T positions in one-chunk (matrix) form from the initial state S0:
 *   Lam_i = sum_{j<=i} dt_j A
 *   y_i   = C_i . (e^{Lam_i} S0) + sum_{j<=i} e^{Lam_i-Lam_j} dt_j (C_i . B_j) x_j + D x_i
 *   S_i   = e^{Lam_i} S0 + sum_{j<=i} e^{Lam_i-Lam_j} dt_j x_j (x) B_j                   */
void or_ssd_chunk(const double *S0, int P, int N, int T, const double *dt, double A, double Dh,
                  const double *x, const double *B, const double *C, double *y, double *snaps) {
    double *Lam = (double *)malloc(sizeof(double) * T);
    double run = 0.0;
    for (int i = 0; i < T; ++i) { run += dt[i] * A; Lam[i] = run; }
    for (int i = 0; i < T; ++i) {
        for (int p = 0; p < P; ++p) {
            double acc = 0.0;
            for (int n = 0; n < N; ++n) acc += C[i * N + n] * exp(Lam[i]) * S0[p * N + n];
            for (int j = 0; j <= i; ++j) {
                double cb = 0.0;
                for (int n = 0; n < N; ++n) cb += C[i * N + n] * B[j * N + n];
                acc += exp(Lam[i] - Lam[j]) * dt[j] * cb * x[j * P + p];
            }
            y[i * P + p] = acc + Dh * x[i * P + p];
        }
        double *Si = snaps + (int64_t)i * P * N;
        for (int p = 0; p < P; ++p)
            for (int n = 0; n < N; ++n) {
                double s = exp(Lam[i]) * S0[p * N + n];
                for (int j = 0; j <= i; ++j) s += exp(Lam[i] - Lam[j]) * dt[j] * x[j * P + p] * B[j * N + n];
                Si[p * N + n] = s;
            }
    }
    free(Lam);
}

/* Gated DeltaNet for one head, S[dv][dk]:
 *   S' = alpha S ; r = S' k ; S = S' + beta (v - r) k^T ; o = S q / sqrt(dk) */
void or_gdn_step(double *S, int dv, int dk, double alpha, double beta,
                 const double *q, const double *k, const double *v, double *o) {
    double sc = 1.0 / sqrt((double)dk);
    for (int i = 0; i < dv; ++i) {
        double *row = S + i * dk;
        double r = 0.0;
        for (int j = 0; j < dk; ++j) { row[j] *= alpha; r += row[j] * k[j]; }
        double u = beta * (v[i] - r), acc = 0.0;
        for (int j = 0; j < dk; ++j) { row[j] += u * k[j]; acc += row[j] * q[j]; }
        o[i] = acc * sc;
    }
}

/* rotate-half RoPE at absolute position pos: pair (i, i+hd/2), frequency theta^(-2i/hd) */
void or_rope(double *x, int hd, int pos, double theta) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow(theta, -2.0 * i / hd);
        double c = cos(ang), s = sin(ang), a = x[i], b = x[i + half];
        x[i] = a * c - b * s;
        x[i + half] = b * c + a * s;
    }
}

/* softmax attention of one query position over rows 0..len-1, grouped-query heads */
void or_attention(const double *q, const uint16_t *Kb, const uint16_t *Vb, int64_t row_stride,
                  int len, int qh, int kvh, int hd, double *out) {
    int group = qh / kvh;
    double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel for schedule(static) if (len * hd > 16384)
    for (int h = 0; h < qh; ++h) {
        int kh = h / group;
        double *p = (double *)malloc(sizeof(double) * len);
        double mx = -INFINITY;
        for (int r = 0; r < len; ++r) {
            const uint16_t *kr = Kb + r * row_stride + kh * hd;
            double s = 0.0;
            for (int e = 0; e < hd; ++e) s += q[h * hd + e] * bf16_val(kr[e]);
            p[r] = s * scale;
            if (p[r] > mx) mx = p[r];
        }
        double den = 0.0;
        for (int r = 0; r < len; ++r) { p[r] = exp(p[r] - mx); den += p[r]; }
        for (int e = 0; e < hd; ++e) {
            double acc = 0.0;
            for (int r = 0; r < len; ++r) acc += p[r] * bf16_val(Vb[r * row_stride + kh * hd + e]);
            out[h * hd + e] = acc / den;
        }
        free(p);
    }
}

int or_argmax_margin(const double *logits, int V, double *margin) {
    int best = 0; float b1 = (float)logits[0], b2 = -INFINITY;
    for (int i = 1; i < V; ++i) {
        float v = (float)logits[i];
        if (v > b1) { b2 = b1; b1 = v; best = i; }
        else if (v > b2) b2 = v;
    }
    if (margin) *margin = (double)b1 - (double)b2;
    return best;
}

int or_accept_len(const int *d, const int *g, int k) {
    int n = 0;
    while (n < k && d[n] == g[n]) ++n;
    return n;
}

/* -------------------------------------------------------------------- model */
typedef struct { double *ssm, *conv, *gdn; } rstate;

struct or_model {
    or_config c; const uint8_t *blob; or_layer *layers;
    int *plan;                          /* per-layer draft plan (OR_DRAFT_*), NULL = the component-aware draft */
    int literal;                        /* 1: M_S keeps a recurrent state of its own over the whole history (Eq. 4 / Eq. 5 read literally) */
    int64_t embed, lm_head, final_norm;
    int64_t n_ssm, n_conv, n_gdn;       /* doubles per sequence */
    int convd;
};

struct or_seq {
    or_model *m; rstate st; uint16_t *K, *V; int len, pending;
    rstate std;                         /* the draft model's own state (literal reading), having consumed the same len tokens */
};

static const float *fvec(const or_model *m, int64_t off) { return (const float *)(m->blob + off); }

or_model *or_model_create(const or_config *c, const uint8_t *blob, const or_layer *layers,
                          int64_t embed, int64_t lm_head, int64_t final_norm) {
    or_model *m = (or_model *)calloc(1, sizeof(or_model));
    m->c = *c; m->blob = blob;
    m->layers = (or_layer *)malloc(sizeof(or_layer) * c->L);
    memcpy(m->layers, layers, sizeof(or_layer) * c->L);
    m->embed = embed; m->lm_head = lm_head; m->final_norm = final_norm;
    if (c->arch == 0) { m->convd = c->H * c->P + 2 * c->N; m->n_ssm = (int64_t)c->L * c->H * c->P * c->N; }
    else { m->convd = 2 * c->gh * c->gdk + c->gh * c->gdv; m->n_gdn = (int64_t)c->L * c->gh * c->gdv * c->gdk; }
    m->n_conv = (int64_t)c->L * (c->conv_w - 1) * m->convd;
    return m;
}
void or_model_destroy(or_model *m) { if (m) { free(m->layers); free(m->plan); free(m); } }

/* Draft strategies (paper Sec. 4.2): which layers the draft model M_S runs.  plan[l] = OR_DRAFT_SKIP: the layer is
 * the identity (layer skipping, "LayerSkip"); OR_DRAFT_LINEAR: only the SSM / linear-attention pathway (Eq. 4; an
 * attention layer of a sequential hybrid is then the identity, Eq. 5); OR_DRAFT_FULL: the whole layer, attention
 * included.  NULL restores the component-aware draft (every layer OR_DRAFT_LINEAR). */
void or_model_set_draft_plan(or_model *m, const int *plan) {
    free(m->plan); m->plan = NULL;
    if (plan) { m->plan = (int *)malloc(sizeof(int) * m->c.L); memcpy(m->plan, plan, sizeof(int) * m->c.L); }
}

static void rstate_alloc(const or_model *m, rstate *s) {
    s->ssm = m->n_ssm ? (double *)calloc(m->n_ssm, sizeof(double)) : NULL;
    s->gdn = m->n_gdn ? (double *)calloc(m->n_gdn, sizeof(double)) : NULL;
    s->conv = (double *)calloc(m->n_conv, sizeof(double));
}
static void rstate_free(rstate *s) { free(s->ssm); free(s->gdn); free(s->conv); }
static void rstate_copy(const or_model *m, rstate *dst, const rstate *src) {
    if (m->n_ssm) memcpy(dst->ssm, src->ssm, sizeof(double) * m->n_ssm);
    if (m->n_gdn) memcpy(dst->gdn, src->gdn, sizeof(double) * m->n_gdn);
    memcpy(dst->conv, src->conv, sizeof(double) * m->n_conv);
}

static int64_t kv_elems(const or_model *m) {
    return (int64_t)m->c.L * m->c.kv_capacity * m->c.kvh * m->c.hd;
}
or_seq *or_seq_create(or_model *m) {
    or_seq *s = (or_seq *)calloc(1, sizeof(or_seq));
    s->m = m; rstate_alloc(m, &s->st); rstate_alloc(m, &s->std);
    s->K = (uint16_t *)calloc(kv_elems(m), 2);
    s->V = (uint16_t *)calloc(kv_elems(m), 2);
    s->pending = -1;
    return s;
}
void or_seq_destroy(or_seq *s) { if (s) { rstate_free(&s->st); rstate_free(&s->std); free(s->K); free(s->V); free(s); } }
void or_seq_reset(or_seq *s) {
    const or_model *m = s->m;
    if (m->n_ssm) memset(s->st.ssm, 0, sizeof(double) * m->n_ssm);
    if (m->n_gdn) memset(s->st.gdn, 0, sizeof(double) * m->n_gdn);
    memset(s->st.conv, 0, sizeof(double) * m->n_conv);
    if (m->n_ssm) memset(s->std.ssm, 0, sizeof(double) * m->n_ssm);
    if (m->n_gdn) memset(s->std.gdn, 0, sizeof(double) * m->n_gdn);
    memset(s->std.conv, 0, sizeof(double) * m->n_conv);
    s->len = 0; s->pending = -1;
}
int or_seq_len(const or_seq *s) { return s->len; }
int or_seq_pending(const or_seq *s) { return s->pending; }
void or_seq_set(or_seq *s, int len, int pending) { s->len = len; s->pending = pending; }
double *or_seq_ssm(or_seq *s) { return s->st.ssm; }
double *or_seq_conv(or_seq *s) { return s->st.conv; }
double *or_seq_gdn(or_seq *s) { return s->st.gdn; }
double *or_seq_draft_ssm(or_seq *s) { return s->std.ssm; }
double *or_seq_draft_conv(or_seq *s) { return s->std.conv; }
double *or_seq_draft_gdn(or_seq *s) { return s->std.gdn; }
uint16_t *or_seq_k(or_seq *s) { return s->K; }
uint16_t *or_seq_v(or_seq *s) { return s->V; }

/* h <- h + W_down( silu(W_gate u) * (W_up u) ), u = rmsnorm(h; norm2) */
static void mlp_block(const or_model *m, const or_layer *ly, double *h) {
    const or_config *c = &m->c;
    double *u = (double *)malloc(sizeof(double) * c->d);
    double *g = (double *)malloc(sizeof(double) * c->ff);
    double *up = (double *)malloc(sizeof(double) * c->ff);
    double *o = (double *)malloc(sizeof(double) * c->d);
    or_rmsnorm(h, fvec(m, ly->norm2), c->d, c->eps, u);
    or_matvec(m->blob, ly->Wgate, c->ff, c->d, u, g);
    or_matvec(m->blob, ly->Wup, c->ff, c->d, u, up);
    for (int i = 0; i < c->ff; ++i) g[i] = silu(g[i]) * up[i];
    or_matvec(m->blob, ly->Wdown, c->d, c->ff, g, o);
    for (int i = 0; i < c->d; ++i) h[i] += o[i];
    free(u); free(g); free(up); free(o);
}

/* f_attn(u): projections, RoPE at pos, append row pos to the cache, attend over rows 0..pos, W_o */
static void attn_branch(const or_model *m, const or_layer *ly, int l, or_seq *s, int pos,
                        const double *u, double *out /* d */) {
    const or_config *c = &m->c;
    int nq = c->qh * c->hd, nkv = c->kvh * c->hd;
    double *q = (double *)malloc(sizeof(double) * nq);
    double *k = (double *)malloc(sizeof(double) * nkv);
    double *v = (double *)malloc(sizeof(double) * nkv);
    double *o = (double *)malloc(sizeof(double) * nq);
    or_matvec(m->blob, ly->Wq, nq, c->d, u, q);
    or_matvec(m->blob, ly->Wk, nkv, c->d, u, k);
    or_matvec(m->blob, ly->Wv, nkv, c->d, u, v);
    for (int h = 0; h < c->qh; ++h) or_rope(q + h * c->hd, c->hd, pos, c->rope_theta);
    for (int h = 0; h < c->kvh; ++h) or_rope(k + h * c->hd, c->hd, pos, c->rope_theta);
    int64_t lbase = (int64_t)l * c->kv_capacity * nkv;
    uint16_t *Kl = s->K + lbase, *Vl = s->V + lbase;
    for (int e = 0; e < nkv; ++e) { Kl[(int64_t)pos * nkv + e] = to_bf16(k[e]); Vl[(int64_t)pos * nkv + e] = to_bf16(v[e]); }
    or_attention(q, Kl, Vl, nkv, pos + 1, c->qh, c->kvh, c->hd, o);
    or_matvec(m->blob, ly->Wo, c->d, nq, o, out);
    free(q); free(k); free(v); free(o);
}

/* f_ssm(u): in-projection, conv + SiLU, softplus(dt), recurrence, gate, gated RMSNorm, W_out */
static void ssm_branch(const or_model *m, const or_layer *ly, int l, rstate *st, const double *u, double *out) {
    const or_config *c = &m->c;
    int di = c->H * c->P, convd = m->convd, N = c->N;
    double *z = (double *)malloc(sizeof(double) * di);
    double *xbc = (double *)malloc(sizeof(double) * convd);
    double *dt = (double *)malloc(sizeof(double) * c->H);
    double *y = (double *)malloc(sizeof(double) * di);
    or_matvec(m->blob, ly->Wz, di, c->d, u, z);
    or_matvec(m->blob, ly->Wxbc, convd, c->d, u, xbc);
    or_matvec(m->blob, ly->Wdt, c->H, c->d, u, dt);
    const float *cw = fvec(m, ly->conv_w), *cb = fvec(m, ly->conv_b);
    double *win = st->conv + (int64_t)l * (c->conv_w - 1) * convd;   /* [3][convd] */
    for (int ch = 0; ch < convd; ++ch) {
        double w3[3] = { win[ch], win[convd + ch], win[2 * convd + ch] };
        double pre = or_conv_step(w3, xbc[ch], cw + ch * 4, cb[ch]);
        win[ch] = w3[0]; win[convd + ch] = w3[1]; win[2 * convd + ch] = w3[2];
        xbc[ch] = silu(pre);
    }
    const double *x = xbc, *B = xbc + di, *C = xbc + di + N;
    const float *A_log = fvec(m, ly->A_log), *Dv = fvec(m, ly->D), *dtb = fvec(m, ly->dt_bias);
    for (int h = 0; h < c->H; ++h) {
        double dth = softplus(dt[h] + dtb[h]);
        double A = -exp((double)A_log[h]);
        double *S = st->ssm + ((int64_t)l * c->H + h) * c->P * N;
        or_ssm_step(S, c->P, N, dth, A, Dv[h], x + h * c->P, B, C, y + h * c->P);
    }
    for (int i = 0; i < di; ++i) y[i] *= silu(z[i]);
    or_rmsnorm(y, fvec(m, ly->gnorm), di, c->eps, z);
    or_matvec(m->blob, ly->Wout, c->d, di, z, out);
    free(z); free(xbc); free(dt); free(y);
}

/* f_lin(u) for a Gated DeltaNet layer */
static void gdn_branch(const or_model *m, const or_layer *ly, int l, rstate *st, const double *u, double *out) {
    const or_config *c = &m->c;
    int nk = c->gh * c->gdk, nv = c->gh * c->gdv, convd = m->convd;
    double *qkv = (double *)malloc(sizeof(double) * convd);
    double *z = (double *)malloc(sizeof(double) * nv);
    double *ga = (double *)malloc(sizeof(double) * c->gh);
    double *gb = (double *)malloc(sizeof(double) * c->gh);
    double *o = (double *)malloc(sizeof(double) * nv);
    or_matvec(m->blob, ly->Wq, nk, c->d, u, qkv);
    or_matvec(m->blob, ly->Wk, nk, c->d, u, qkv + nk);
    or_matvec(m->blob, ly->Wv, nv, c->d, u, qkv + 2 * nk);
    or_matvec(m->blob, ly->Wgz, nv, c->d, u, z);
    or_matvec(m->blob, ly->Wga, c->gh, c->d, u, ga);
    or_matvec(m->blob, ly->Wgb, c->gh, c->d, u, gb);
    const float *cw = fvec(m, ly->conv_w), *cb = fvec(m, ly->conv_b);
    double *win = st->conv + (int64_t)l * (c->conv_w - 1) * convd;
    for (int ch = 0; ch < convd; ++ch) {
        double w3[3] = { win[ch], win[convd + ch], win[2 * convd + ch] };
        double pre = or_conv_step(w3, qkv[ch], cw + ch * 4, cb[ch]);
        win[ch] = w3[0]; win[convd + ch] = w3[1]; win[2 * convd + ch] = w3[2];
        qkv[ch] = silu(pre);
    }
    const float *onw = fvec(m, ly->gnorm);
    for (int h = 0; h < c->gh; ++h) {
        double *q = qkv + h * c->gdk, *k = qkv + nk + h * c->gdk, *v = qkv + 2 * nk + h * c->gdv;
        double nq = 0.0, nkk = 0.0;
        for (int j = 0; j < c->gdk; ++j) { nq += q[j] * q[j]; nkk += k[j] * k[j]; }
        nq = 1.0 / sqrt(nq + 1e-6); nkk = 1.0 / sqrt(nkk + 1e-6);
        for (int j = 0; j < c->gdk; ++j) { q[j] *= nq; k[j] *= nkk; }
        double *S = st->gdn + ((int64_t)l * c->gh + h) * c->gdv * c->gdk;
        double *oh = o + h * c->gdv;
        or_gdn_step(S, c->gdv, c->gdk, sigmoid(ga[h]), sigmoid(gb[h]), q, k, v, oh);
        or_rmsnorm(oh, onw, c->gdv, c->eps, oh);
        for (int i = 0; i < c->gdv; ++i) oh[i] *= silu(z[h * c->gdv + i]);
    }
    or_matvec(m->blob, ly->Wout, c->d, nv, o, out);
    free(qkv); free(z); free(ga); free(gb); free(o);
}

/* One token through the stack.  mode 0: full model M_H (Eq. 2 / Eq. 3); mode 1: draft M_S
 * (Eq. 4: attention output zeroed; Eq. 5: attention layers are the identity; or the model's per-layer draft plan,
 * Sec. 4.2: layers skipped as a whole, layers kept whole).  A draft layer that runs attention writes its K/V row at
 * `pos`, beyond the committed length: scratch rows that the verification pass overwrites. */
static void model_step(const or_model *m, or_seq *s, rstate *st, int token, int pos, int mode, double *logits) {
    const or_config *c = &m->c;
    int d = c->d;
    double *h = (double *)malloc(sizeof(double) * d);
    double *u = (double *)malloc(sizeof(double) * d);
    double *a = (double *)malloc(sizeof(double) * d);
    const uint16_t *e = (const uint16_t *)(m->blob + m->embed) + (int64_t)token * d;
    for (int i = 0; i < d; ++i) h[i] = bf16_val(e[i]);
    for (int l = 0; l < c->L; ++l) {
        const or_layer *ly = &m->layers[l];
        /* what this layer does in this pass: the full model runs every layer whole; the draft follows its plan */
        const int what = mode == 0 ? OR_DRAFT_FULL : (m->plan ? m->plan[l] : OR_DRAFT_LINEAR);
        if (what == OR_DRAFT_SKIP) continue;                         /* h_l = h_{l-1} */
        if (ly->type == 0) {
            or_rmsnorm(h, fvec(m, ly->norm1), d, c->eps, u);
            ssm_branch(m, ly, l, st, u, a);
            if (what == OR_DRAFT_FULL) {
                double *b = (double *)malloc(sizeof(double) * d);
                attn_branch(m, ly, l, s, pos, u, b);
                for (int i = 0; i < d; ++i) a[i] += b[i];
                free(b);
            }
            for (int i = 0; i < d; ++i) h[i] += a[i];
            mlp_block(m, ly, h);
        } else if (ly->type == 1) {
            or_rmsnorm(h, fvec(m, ly->norm1), d, c->eps, u);
            gdn_branch(m, ly, l, st, u, a);
            for (int i = 0; i < d; ++i) h[i] += a[i];
            mlp_block(m, ly, h);
        } else {
            if (what != OR_DRAFT_FULL) continue;            /* h_l = h_{l-1} */
            or_rmsnorm(h, fvec(m, ly->norm1), d, c->eps, u);
            attn_branch(m, ly, l, s, pos, u, a);
            for (int i = 0; i < d; ++i) h[i] += a[i];
            mlp_block(m, ly, h);
        }
    }
    or_rmsnorm(h, fvec(m, m->final_norm), d, c->eps, u);
    or_mat Wlm = { m->lm_head, d };
    or_matvec(m->blob, Wlm, c->V, d, u, logits);
    free(h); free(u); free(a);
}

/* Whose recurrent state the draft starts from.  0 (default): every round M_S starts from the committed state of the full
 * model (shared state).  1: Eq. 4 / Eq. 5 read literally - h^S is computed from h^S at every position, so M_S has a
 * recurrent state of its own that has seen the whole history without attention; it advances over exactly the tokens
 * the sequence consumes.  The emitted tokens are the same under both readings (greedy verification is lossless). */
void or_model_set_literal_draft(or_model *m, int on) { m->literal = on != 0; }

int or_step_committed(or_seq *s, int token, int mode, double *logits) {
    if (mode == 0 && s->len >= s->m->c.kv_capacity) return -1;
    if (mode == 0 && s->m->literal) {       /* the draft model consumes the token too, on its own state */
        double *lg = (double *)malloc(sizeof(double) * s->m->c.V);
        model_step(s->m, s, &s->std, token, s->len, 1, lg);
        free(lg);
    }
    model_step(s->m, s, (mode == 1 && s->m->literal) ? &s->std : &s->st, token, s->len, mode, logits);
    if (mode == 0) s->len += 1;
    return 0;
}

int or_prefill(or_seq *s, const int *tokens, int n) {
    if (n < 1 || s->len + n > s->m->c.kv_capacity) return -1;
    double *lg = (double *)malloc(sizeof(double) * s->m->c.V);
    for (int i = 0; i < n; ++i) or_step_committed(s, tokens[i], 0, lg);
    s->pending = or_argmax_margin(lg, s->m->c.V, NULL);
    free(lg);
    return 0;
}

int or_greedy(or_seq *s, int n, int *out) {
    if (s->pending < 0 || s->len + n > s->m->c.kv_capacity) return -1;
    double *lg = (double *)malloc(sizeof(double) * s->m->c.V);
    for (int i = 0; i < n; ++i) {
        out[i] = s->pending;
        or_step_committed(s, s->pending, 0, lg);
        s->pending = or_argmax_margin(lg, s->m->c.V, NULL);
    }
    free(lg);
    return 0;
}

int or_draft_only(or_seq *s, int k, int *d, double *logits) {
    const or_model *m = s->m;
    rstate scratch; rstate_alloc(m, &scratch); rstate_copy(m, &scratch, m->literal ? &s->std : &s->st);
    double *lg = (double *)malloc(sizeof(double) * m->c.V);
    int tok = s->pending;
    for (int i = 0; i < k; ++i) {
        model_step(m, s, &scratch, tok, s->len + i, 1, lg);
        if (logits) memcpy(logits + (int64_t)i * m->c.V, lg, sizeof(double) * m->c.V);
        tok = d[i] = or_argmax_margin(lg, m->c.V, NULL);
    }
    free(lg); rstate_free(&scratch);
    return 0;
}

int or_round(or_seq *s, int k, const int *cand_in, int forced_n, int forced_next,
             int *cand_o, int *g_o, double *margin_o, double *logits_o, int *n_acc, int *emitted) {
    const or_model *m = s->m;
    int T = k + 1, V = m->c.V;
    if (k < 0 || s->len + T > m->c.kv_capacity) return -1;
    if (!cand_in && s->pending < 0) return -2;
    if (forced_n > k) return -3;
    int *cand = (int *)malloc(sizeof(int) * T), *g = (int *)malloc(sizeof(int) * T);
    double *lg = (double *)malloc(sizeof(double) * V);
    /* draft phase: M_S proposes k tokens from a scratch copy of the committed state */
    if (cand_in) memcpy(cand, cand_in, sizeof(int) * T);
    else { cand[0] = s->pending; or_draft_only(s, k, cand + 1, NULL); }
    /* verification phase: M_H over the T candidates, one literal step each, keeping every state */
    rstate *snap = (rstate *)malloc(sizeof(rstate) * T);
    rstate run; rstate_alloc(m, &run); rstate_copy(m, &run, &s->st);
    for (int i = 0; i < T; ++i) {
        model_step(m, s, &run, cand[i], s->len + i, 0, lg);
        double mg; g[i] = or_argmax_margin(lg, V, &mg);
        if (margin_o) margin_o[i] = mg;
        if (logits_o) memcpy(logits_o + (int64_t)i * V, lg, sizeof(double) * V);
        rstate_alloc(m, &snap[i]); rstate_copy(m, &snap[i], &run);
    }
    /* greedy acceptance: draft i+1 is kept iff it equals the full model's choice g[i] */
    int n = forced_n >= 0 ? forced_n : or_accept_len(cand + 1, g, k);
    int next = forced_next >= 0 ? forced_next : g[n];
    if (emitted) { for (int i = 0; i < n; ++i) emitted[i] = cand[i + 1]; emitted[n] = next; }
    /* literal reading: the draft model's own state advances over exactly the consumed tokens c_0 .. c_n */
    if (m->literal)
        for (int i = 0; i <= n; ++i) model_step(m, s, &s->std, cand[i], s->len + i, 1, lg);
    /* rollback: state after the accepted prefix; rows beyond it in the cache are dead */
    rstate_copy(m, &s->st, &snap[n]);
    s->len += n + 1; s->pending = next;
    if (n_acc) *n_acc = n;
    if (cand_o) memcpy(cand_o, cand, sizeof(int) * T);
    if (g_o) memcpy(g_o, g, sizeof(int) * T);
    for (int i = 0; i < T; ++i) rstate_free(&snap[i]);
    rstate_free(&run); free(snap); free(cand); free(g); free(lg);
    return 0;
}


/* ------------------------------------------------- speculative sampling at temperature > 0 (paper Sec. 3.3, Eq. 6) */
/* p_j = exp((l_j - max l) / tau) / Z */
void or_softmax_t(const double *logits, int V, double tau, double *p) {
    double mx = logits[0];
    for (int j = 1; j < V; ++j) if (logits[j] > mx) mx = logits[j];
    double Z = 0.0;
    for (int j = 0; j < V; ++j) { p[j] = exp((logits[j] - mx) / tau); Z += p[j]; }
    for (int j = 0; j < V; ++j) p[j] /= Z;
}

/* Inverse-CDF draw from unnormalised non-negative weights: the smallest j whose cumulative weight exceeds u * total
 * (u in [0,1)).  *margin: distance of the threshold to the nearer cumulative boundary of j, relative to the total
 * (how far u is from choosing a neighbour).  Total 0: returns -1. */
int or_sample_cdf(const double *w, int V, double u, double *margin) {
    double tot = 0.0;
    for (int j = 0; j < V; ++j) tot += w[j];
    if (!(tot > 0.0)) { if (margin) *margin = 0.0; return -1; }
    double t = u * tot, c = 0.0;
    int pick = -1; double lo = 0.0, hi = 0.0;
    for (int j = 0; j < V; ++j) {
        double cn = c + w[j];
        if (w[j] > 0.0 && cn > t) { pick = j; lo = c; hi = cn; break; }
        c = cn;
    }
    if (pick < 0) {                       /* u * total rounded up to the total: the last positive weight */
        for (int j = V - 1; j >= 0; --j) if (w[j] > 0.0) { pick = j; break; }
        if (margin) *margin = 0.0;
        return pick;
    }
    if (margin) { double a = t - lo, b = hi - t; *margin = (a < b ? a : b) / tot; }
    return pick;
}

/* Eq. 6: draft token x is accepted with probability min(1, P_H(x) / P_S(x)): accepted iff u < that ratio.
 * *margin = |u - min(1, ratio)| (0 when the ratio is >= 1: then every u accepts and the margin is reported as 1). */
int or_spec_accept(const double *pS, const double *pH, int x, double u, double *margin) {
    double ratio = pS[x] > 0.0 ? pH[x] / pS[x] : 1.0;
    if (ratio >= 1.0) { if (margin) *margin = 1.0; return 1; }
    if (margin) *margin = fabs(u - ratio);
    return u < ratio;
}

/* unnormalised residual distribution max(0, P_H - P_S) a rejected position is resampled from */
void or_residual(const double *pS, const double *pH, int V, double *r) {
    for (int j = 0; j < V; ++j) { double d = pH[j] - pS[j]; r[j] = d > 0.0 ? d : 0.0; }
}

/* One round at temperature tau > 0.  u_draft[k]: uniforms of the k draft draws; u_acc[k]: of the accept tests;
 * u_final: of the correction draw (from the residual at the first rejection) or the bonus draw (from P_H after the
 * last draft when all are accepted).  cand_in (k+1 tokens) replaces pending and the drafts (the draft model is still
 * run over them, for P_S).  margins[2k+1]: draft draws, accept tests (1 where not evaluated), final draw. */
int or_round_sampled(or_seq *s, int k, double tau, const double *u_draft, const double *u_acc, double u_final,
                     const int *cand_in, int forced_n, int forced_next,
                     int *cand_o, int *n_acc, int *emitted, double *margins) {
    const or_model *m = s->m;
    int T = k + 1, V = m->c.V;
    if (k < 0 || !(tau > 0.0) || s->len + T > m->c.kv_capacity) return -1;
    if (!cand_in && s->pending < 0) return -2;
    if (forced_n > k) return -3;
    int *cand = (int *)malloc(sizeof(int) * T);
    double *lg = (double *)malloc(sizeof(double) * V);
    double *pS = (double *)malloc(sizeof(double) * (size_t)(k > 0 ? k : 1) * V);
    double *pH = (double *)malloc(sizeof(double) * (size_t)T * V);
    double *r = (double *)malloc(sizeof(double) * V);
    for (int i = 0; i < 2 * k + 1; ++i) margins[i] = 1.0;
    /* draft phase: M_S draws k tokens from its own distributions, on a scratch copy of the committed state */
    rstate scratch; rstate_alloc(m, &scratch); rstate_copy(m, &scratch, m->literal ? &s->std : &s->st);
    cand[0] = cand_in ? cand_in[0] : s->pending;
    for (int i = 0; i < k; ++i) {
        model_step(m, s, &scratch, cand[i], s->len + i, 1, lg);
        or_softmax_t(lg, V, tau, pS + (size_t)i * V);
        int tok = or_sample_cdf(pS + (size_t)i * V, V, u_draft[i], &margins[i]);
        cand[i + 1] = cand_in ? cand_in[i + 1] : tok;
        if (cand_in) margins[i] = 1.0;
    }
    rstate_free(&scratch);
    /* verification phase: M_H over the T candidates */
    rstate *snap = (rstate *)malloc(sizeof(rstate) * T);
    rstate run; rstate_alloc(m, &run); rstate_copy(m, &run, &s->st);
    for (int i = 0; i < T; ++i) {
        model_step(m, s, &run, cand[i], s->len + i, 0, lg);
        or_softmax_t(lg, V, tau, pH + (size_t)i * V);
        rstate_alloc(m, &snap[i]); rstate_copy(m, &snap[i], &run);
    }
    /* Eq. 6: accept draft i+1 with probability min(1, P_H / P_S); stop at the first rejection */
    int n = 0;
    while (n < k && or_spec_accept(pS + (size_t)n * V, pH + (size_t)n * V, cand[n + 1], u_acc[n], &margins[k + n])) ++n;
    if (forced_n >= 0) n = forced_n;
    int next;
    if (n < k) { or_residual(pS + (size_t)n * V, pH + (size_t)n * V, V, r); next = or_sample_cdf(r, V, u_final, &margins[2 * k]); }
    else next = or_sample_cdf(pH + (size_t)k * V, V, u_final, &margins[2 * k]);
    if (next < 0) next = or_sample_cdf(pH + (size_t)n * V, V, u_final, &margins[2 * k]);   /* empty residual (P_H <= P_S everywhere, i.e. equal): P_H itself */
    if (forced_next >= 0) next = forced_next;
    if (emitted) { for (int i = 0; i < n; ++i) emitted[i] = cand[i + 1]; emitted[n] = next; }
    if (m->literal)
        for (int i = 0; i <= n; ++i) model_step(m, s, &s->std, cand[i], s->len + i, 1, lg);
    rstate_copy(m, &s->st, &snap[n]);
    s->len += n + 1; s->pending = next;
    if (n_acc) *n_acc = n;
    if (cand_o) memcpy(cand_o, cand, sizeof(int) * T);
    for (int i = 0; i < T; ++i) rstate_free(&snap[i]);
    rstate_free(&run); free(snap); free(cand); free(lg); free(pS); free(pH); free(r);
    return 0;
}

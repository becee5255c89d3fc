/*
 * CPU oracle for component-aware self-speculative decoding on hybrid models.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, double-precision
 * restatement of what the decode path computes: the hybrid block in its two
 * modes (paper Eq. 2-5), the draft / verify / accept round (paper Sec. 3.3)
 * and plain greedy decoding, which the round must reproduce token for token.
 * It shares no code with the CUDA library; only tests, the smoke check and the
 * benchmark's cpu_baseline leg may call it.
 *
 * Parity status: every component and the whole loop are pinned by closed forms,
 * special cases and invariants (see tests).  The absolute logits of the
 * random-init models have no printed value in the paper to compare with:
 * for those, "parity unpinned" - they are only compared oracle <-> GPU.
 *
 * Weights are bf16 bit patterns (exactly representable in double); every
 * other quantity is double.  The KV cache stores bf16-rounded rows because the
 * workload fixes a bf16 KV cache.  Greedy decisions (argmax, top-2 margin) are
 * taken on the logits rounded to float32, the precision the GPU path decides in.
 */
#ifndef HS_ORACLE_H
#define HS_ORACLE_H
#include <stdint.h>

typedef struct {
    int arch;            /* 0 parallel hybrid (Eq. 2), 1 sequential hybrid (Eq. 3) */
    int L, d, V;
    int H, P, N;         /* Mamba-2: heads, head dim, state dim (one B/C group) */
    int conv_w;          /* causal depthwise conv width (4) */
    int qh, kvh, hd;     /* attention */
    int ff;              /* SwiGLU width */
    int gh, gdk, gdv;    /* Gated DeltaNet heads, key dim, value dim */
    int kv_capacity;
    double rope_theta, eps;
} or_config;

typedef struct { int64_t off; int64_t stride; } or_mat;   /* byte offset of row 0, row stride in elements */

typedef struct {
    int type;            /* 0 parallel block, 1 Gated DeltaNet layer, 2 attention layer */
    int64_t norm1, conv_w, conv_b, A_log, D, dt_bias, gnorm, norm2;   /* byte offsets of fp32 vectors, -1 if absent */
    or_mat Wz, Wxbc, Wdt;          /* Mamba in-projection row blocks */
    or_mat Wq, Wk, Wv, Wo;         /* attention (or DeltaNet q,k,v) */
    or_mat Wgz, Wga, Wgb;          /* DeltaNet output gate, decay gate, beta */
    or_mat Wout;                   /* Mamba / DeltaNet out-projection */
    or_mat Wgate, Wup, Wdown;      /* SwiGLU */
} or_layer;

enum { OR_DRAFT_SKIP = 0, OR_DRAFT_LINEAR = 1, OR_DRAFT_FULL = 2 };   /* per-layer draft plan, paper Sec. 4.2 */

typedef struct or_model or_model;
typedef struct or_seq or_seq;

/* ---- component functions (also used by the model step; exported for pins) ---- */
void or_rmsnorm(const double *x, const float *w, int n, double eps, double *out);
void or_matvec(const uint8_t *blob, or_mat W, int rows, int cols, const double *x, double *y);
/* one conv channel: window = 3 cached inputs + cur; returns pre-activation; shifts the window */
double or_conv_step(double *win3, double cur, const float *taps4, double bias);
/* Mamba-2 recurrence, one head: S[P][N] updated in place, y[P] out */
void or_ssm_step(double *S, int P, int N, double dt, double A, double Dh,
                 const double *x, const double *B, const double *C, double *y);
/* one-chunk SSD form from S0 for T positions; snaps[T][P][N], y[T][P] */
void or_ssd_chunk(const double *S0, int P, int N, int T, const double *dt, double A, double Dh,
                  const double *x, const double *B, const double *C, double *y, double *snaps);
/* Gated DeltaNet, one head: S[dv][dk] in place; q,k already L2-normalised; o[dv] out */
void or_gdn_step(double *S, int dv, int dk, double alpha, double beta,
                 const double *q, const double *k, const double *v, double *o);
void or_rope(double *x, int hd, int pos, double theta);
/* one query position: q[qh][hd]; K,V bf16 rows r at Kb + r*row_stride (elements), head h at +h*hd */
void or_attention(const double *q, const uint16_t *Kb, const uint16_t *Vb, int64_t row_stride,
                  int len, int qh, int kvh, int hd, double *out);
/* argmax (lowest index on ties) and top1-top2 margin of logits rounded to float32 */
int or_argmax_margin(const double *logits, int V, double *margin);
/* n = number of leading i<k with d[i]==g[i] */
int or_accept_len(const int *d, const int *g, int k);

/* ---- model and sequence ---- */
or_model *or_model_create(const or_config *c, const uint8_t *blob, const or_layer *layers,
                          int64_t embed, int64_t lm_head, int64_t final_norm);
void or_model_destroy(or_model *m);
/* per-layer draft plan (OR_DRAFT_*), length L; NULL: the component-aware draft of Eq. 4 / Eq. 5 */
void or_model_set_draft_plan(or_model *m, const int *plan);
/* 1: the draft model keeps its own attention-free recurrent state over the whole history (Eq. 4 / Eq. 5 read literally);
 * 0 (default): the draft starts every round from the full model's committed state */
void or_model_set_literal_draft(or_model *m, int on);
or_seq *or_seq_create(or_model *m);
void or_seq_destroy(or_seq *s);
void or_seq_reset(or_seq *s);
int or_seq_len(const or_seq *s);
int or_seq_pending(const or_seq *s);
void or_seq_set(or_seq *s, int len, int pending);
/* raw pointers into the committed state, for export / injection (NULL if the arch has none) */
double *or_seq_ssm(or_seq *s);      /* [L][H][P][N] */
double *or_seq_conv(or_seq *s);     /* [L][conv_w-1][convd] */
double *or_seq_gdn(or_seq *s);      /* [L][gh][gdv][gdk] */
double *or_seq_draft_ssm(or_seq *s);   /* the draft model's own state (literal reading), same layouts */
double *or_seq_draft_conv(or_seq *s);
double *or_seq_draft_gdn(or_seq *s);
uint16_t *or_seq_k(or_seq *s);      /* [L][cap][kvh][hd] bf16 bits */
uint16_t *or_seq_v(or_seq *s);

/* one token through the model on the committed state. mode 0 = full (Eq. 2/3, appends KV row `len`),
 * 1 = draft (Eq. 4/5, no KV access).  Advances len in full mode only.  logits[V]. */
int or_step_committed(or_seq *s, int token, int mode, double *logits);
/* consume all prompt tokens with the full model; pending = greedy choice after the last one */
int or_prefill(or_seq *s, const int *tokens, int n);
/* plain greedy decoding of the full model: emits n tokens starting with the pending one */
int or_greedy(or_seq *s, int n, int *out);
/* one draft-verify-accept-rollback round (Sec. 3.3).  cand_in: NULL, or k+1 tokens to verify
 * instead of drafting.  forced_n / forced_next: -1, or overrides of accept length / next pending.
 * Outputs (any may be NULL): cand[k+1], g[k+1], margin[k+1], logits[(k+1)*V], n_acc, emitted[k+1]. */
int or_round(or_seq *s, int k, const int *cand_in, int forced_n, int forced_next,
             int *cand, int *g, double *margin, double *logits, int *n_acc, int *emitted);
/* draft phase only, on a scratch copy: d[k] and (optional) logits[k*V]; committed state untouched */
int or_draft_only(or_seq *s, int k, int *d, double *logits);

/* ---- speculative sampling at temperature > 0 (paper Sec. 3.3, Eq. 6) ---- */
void or_softmax_t(const double *logits, int V, double tau, double *p);
int or_sample_cdf(const double *w, int V, double u, double *margin);
int or_spec_accept(const double *pS, const double *pH, int x, double u, double *margin);
void or_residual(const double *pS, const double *pH, int V, double *r);
int or_round_sampled(or_seq *s, int k, double tau, const double *u_draft, const double *u_acc, double u_final,
                     const int *cand_in, int forced_n, int forced_next,
                     int *cand_o, int *n_acc, int *emitted, double *margins);

#endif

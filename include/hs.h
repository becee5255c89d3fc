/*
 * libhs - decode hot path of component-aware self-speculative decoding on hybrid
 * language models, for one NVIDIA B200 (sm_100a).
 *
 * One speculative round (paper Sec. 3.3) is
 *     hs_draft(k)  ->  hs_verify(k)  ->  hs_accept_rollback()
 * - draft:  the draft model M_S (paper Eq. 4: attention output zeroed in a parallel hybrid;
 *   Eq. 5: attention layers are the identity in a sequential hybrid) proposes k tokens
 *   autoregressively from the committed recurrent state, on scratch state, without touching
 *   the KV cache;
 * - verify: the full model M_H (Eq. 2 / Eq. 3) processes the k+1 candidates in one pass, keeps the
 *   recurrent state after every position and appends k+1 KV rows;
 * - accept/rollback: greedy rule (Sec. 3.3, T = 0): drafts are kept up to the first position whose
 *   draft token differs from the full model's argmax; the committed state becomes the snapshot of
 *   the last accepted position and the KV length is cut to the accepted prefix.
 *
 * Conventions
 * - All functions return HS_OK (0) or a negative hs_status.  Nothing throws, aborts or traps.
 * - The library allocates NO device memory.  Every device buffer is supplied by the caller in
 *   hs_buffers (sizes from hs_query_sizes), must be 256-byte aligned and must outlive the handle.
 *   The library owns only the host-side handle.
 * - All device work is enqueued on the stream given to hs_init_model.  Calls are asynchronous
 *   unless they take or return HOST data (documented per call).
 * - "dev" / "host" in a parameter name says where the pointer must live.
 * - Sequence b (0 <= b < batch) owns: kv_len[b] consumed tokens (KV rows 0..kv_len-1 and the
 *   recurrent state reflect them) and a pending token: the full model's greedy choice after those
 *   tokens, already emitted, not yet consumed.
 */
#ifndef HS_H
#define HS_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HS_OK = 0,
    HS_ERR_INVALID_ARG = -1,  /* null pointer, bad shape, k out of range, ... */
    HS_ERR_SIZE = -2,         /* a caller buffer is smaller than hs_query_sizes reports */
    HS_ERR_CAPACITY = -3,     /* kv_len + k + 1 would exceed kv_capacity */
    HS_ERR_ORDER = -4,        /* call sequence violated (e.g. accept before verify) */
    HS_ERR_CUDA = -5,         /* CUDA runtime error; text in hs_last_error */
    HS_ERR_TIMEOUT = -6,      /* a bounded device-side wait expired */
    HS_ERR_DEVICE = -7        /* a kernel reported an inconsistency through the status word */
} hs_status;

enum { HS_ARCH_PARALLEL = 0, HS_ARCH_SEQUENTIAL = 1 };
/* layer kinds: parallel block (Mamba-2 + attention summed, Eq. 2); Gated DeltaNet layer and
 * attention layer of a sequential hybrid (Eq. 3; layer l is attention iff l % 4 == 3) */
enum { HS_LAYER_PAR = 0, HS_LAYER_GDN = 1, HS_LAYER_ATT = 2 };

typedef struct hs_config {
    int32_t arch;              /* HS_ARCH_* */
    int32_t L, d, V;           /* layers, model width, vocabulary */
    int32_t H, P, N;           /* Mamba-2 heads, head dim, state dim (one B/C group); parallel arch */
    int32_t conv_w;            /* causal depthwise conv width; must be 4 */
    int32_t qh, kvh, hd;       /* attention: query heads, KV heads, head dim */
    int32_t ff;                /* SwiGLU width */
    int32_t gh, gdk, gdv;      /* Gated DeltaNet heads, key dim, value dim; sequential arch */
    int32_t max_batch;         /* sequences resident at once */
    int32_t max_k;             /* largest draft length (<= 8) */
    int32_t kv_capacity;       /* KV rows per sequence */
    float rope_theta;          /* 10000 */
    float eps;                 /* RMSNorm epsilon */
    int32_t flags;             /* HS_FLAG_* */
} hs_config;

enum {
    HS_FLAG_GRAPHS = 1,        /* replay each (mode, k, batch) step as a captured CUDA graph */
    HS_FLAG_REPLAY = 2,        /* rollback by replay: verify keeps no per-position state snapshots but a small log of
                                  the k+1 state updates (Mamba-2: decay, dt*x, B; DeltaNet: alpha, beta, k, v), and
                                  hs_accept_rollback applies the accepted n+1 updates to the committed state in place.
                                  State traffic per verify round: 3 state units (read, read, write) instead of k+2;
                                  the snapshot buffer shrinks to one state per sequence plus the log.  Same results. */
    HS_FLAG_LITERAL_DRAFT = 4  /* whose recurrent state the draft starts from.  Default (flag clear): every round the draft
                                  starts from the committed state of the full model.  With the flag, Eq. 4 / Eq. 5 are read
                                  literally: the draft model M_S keeps a recurrent state and conv window of its own, which have
                                  seen the whole history without attention and advance over exactly the tokens a round
                                  consumes (hs_prefill runs M_S over the prompt as well; a round runs k+1 draft steps, the
                                  last one only to consume d_k).  The emitted tokens are the same (greedy verification is
                                  lossless); the acceptance rate of real weights and the cost of a round differ.  The draft
                                  scratch buffer grows to max_k+2 states per sequence.  Only with draft plans that keep no
                                  attention. */
};

/* Bytes the caller must provide (each buffer 256-byte aligned). */
typedef struct hs_sizes {
    int64_t weights;           /* weight blob, format below */
    int64_t snap;              /* recurrent-state snapshots [rec layer][seq][max_k+1][state] fp32; with HS_FLAG_REPLAY:
                                  committed states [rec layer][seq][state], then the update log [rec layer][seq][max_k+1][w] */
    int64_t dstate;            /* draft scratch state       [rec layer][seq][state] fp32 */
    int64_t conv;              /* conv windows: committed, per-position history, draft ping-pong, fp32 */
    int64_t kv;                /* K then V: [attn layer][seq][kv head][kv_capacity][hd] bf16 each */
    int64_t work;              /* activations, logits, split-KV partials, RoPE table, control block */
} hs_sizes;

typedef struct hs_buffers {    /* DEVICE pointers */
    const void *weights;
    void *snap, *dstate, *conv, *kv, *work;
} hs_buffers;

typedef struct hs_model hs_model;

/*
 * Weight blob format (all offsets multiples of 256 bytes; bf16 matrices are row-major [out, in]).
 * Globals, in order: EMBED [V,d] bf16, LM_HEAD [V,d] bf16, FINAL_NORM [d] f32.
 * Then per layer, the tensors its kind has, in id order:
 *   0 NORM1 [d] f32
 *   1 W_IN  bf16, row blocks:  parallel: z[di] x[di] B[N] C[N] dt[H] q[qh*hd] k[kvh*hd] v[kvh*hd]
 *                              DeltaNet: q[gh*gdk] k[gh*gdk] v[gh*gdv] z[gh*gdv] a[gh] b[gh]
 *                              attention: q k v
 *   2 CONV_W [channels,4] f32 (tap 3 weights the newest input), 3 CONV_B [channels] f32
 *   4 A_LOG [H], 5 D [H], 6 DT_BIAS [H] f32                        (parallel only)
 *   7 GNORM f32: gated-norm weight [di] (parallel) / per-head output-norm weight [gdv] (DeltaNet)
 *   8 W_OUT [d, di] or [d, gh*gdv] bf16, 9 W_O [d, qh*hd] bf16
 *   10 NORM2 [d] f32, 11 W_GU [2*ff, d] bf16 (row 2i = gate_i, row 2i+1 = up_i), 12 W_DOWN [d, ff] bf16
 * hs_weight_offset returns the byte offset of (layer, tensor id), layer = -1 for the globals
 * (ids 0..2), or -1 if the layer has no such tensor.
 */
enum { HS_T_NORM1 = 0, HS_T_W_IN, HS_T_CONV_W, HS_T_CONV_B, HS_T_A_LOG, HS_T_D, HS_T_DT_BIAS, HS_T_GNORM,
       HS_T_W_OUT, HS_T_W_O, HS_T_NORM2, HS_T_W_GU, HS_T_W_DOWN, HS_T_COUNT };
enum { HS_G_EMBED = 0, HS_G_LM_HEAD = 1, HS_G_FINAL_NORM = 2 };

/* Sizes of the caller's buffers for this configuration.  Host only, no CUDA call.
 * HS_ERR_INVALID_ARG if the shape is unsupported (see hs_init_model). */
int hs_query_sizes(const hs_config *cfg, hs_sizes *out);
int64_t hs_weight_offset(const hs_config *cfg, int layer, int tensor);

/* Build the host handle for one hybrid model (paper Sec. 3.1: Eq. 2 parallel block / Eq. 3 sequential stack)
 * and its two modes (Sec. 3.2).  Requirements: conv_w == 4; d, ff, di, qh*hd, gh*gdv multiples of 256;
 * P and gdv multiples of 16; N in {64,128,256}; hd in {64,128}; gdk == 64; qh % kvh == 0;
 * (qh/kvh)*(max_k+1) <= 48; max_k <= 8.
 * bufs: the six DEVICE buffers (caller-owned, 256-byte aligned, alive until hs_destroy); have: the number of
 * bytes the caller really provides in each of them - HS_ERR_SIZE if any is smaller than hs_query_sizes reports.
 * The weights must already be in `bufs->weights` in the blob format.  Enqueues (on `stream`, a cudaStream_t)
 * the RoPE table upload and the zeroing of the control block, and synchronises; does not read the other buffers.
 * On any error *out is set to NULL and nothing is left to destroy. */
int hs_init_model(const hs_config *cfg, const hs_buffers *bufs, const hs_sizes *have, void *stream, hs_model **out);

/* Zero every sequence: recurrent state, conv windows, kv_len = 0, no pending token.  Async. */
int hs_reset(hs_model *m);

/* Consume prompts with the full model (paper Sec. 3.3 prefix x_{1:t}; M_H of Eq. 2 / Eq. 3).  tokens_host: the
 * prompts back to back (sequence b starts at sum(lens_host[0..b-1])); lens_host[b] >= 1; every id in [0, V),
 * otherwise HS_ERR_INVALID_ARG before anything is enqueued.  Sets the batch
 * size for the following rounds.  Afterwards kv_len[b] = lens[b] and pending[b] = the greedy choice
 * after the last prompt token (generated token #1).  Runs as verify passes over chunks of max_k+1 prompt
 * positions, all sequences of equal chunk length together, with every candidate accepted; nothing waits on the host
 * between chunks.  Synchronises the stream before returning (tokens_host may be reused afterwards). */
int hs_prefill(hs_model *m, const int32_t *tokens_host, const int32_t *lens_host, int batch);

/* Draft phase (paper Sec. 3.3, "Draft phase": M_S generates k tokens autoregressively; M_S is Eq. 4 for a
 * parallel hybrid - attention output zeroed - and Eq. 5 for a sequential one - attention layers are the
 * identity): k draft-mode steps for every sequence on scratch state; candidates
 * cand[b][0..k] = [pending, d_1..d_k] stay on the device; the KV cache and the committed state are not touched.
 * 0 <= k <= max_k; k = 0 does nothing.  HS_ERR_ORDER between hs_verify and hs_accept_rollback.  Async. */
int hs_draft(hs_model *m, int k);

/* Draft strategy (paper Sec. 4.2 and Table 8; Sec. 6.2 recommends layer skipping for sequential hybrids): what
 * each layer does in draft mode.  plan_host: int32 [L] on the HOST, or NULL for the component-aware draft (every
 * entry HS_DRAFT_LINEAR).
 *   HS_DRAFT_SKIP    the layer is the identity (mixer and MLP skipped: "LayerSkip")
 *   HS_DRAFT_LINEAR  only the SSM / linear-attention pathway runs (Eq. 4); an attention layer of a sequential
 *                    hybrid is then the identity (Eq. 5)
 *   HS_DRAFT_FULL    the whole layer, attention included.  Such a draft reads the committed KV cache and appends
 *                    its own rows behind it (rows kv_len .. kv_len+k-1: scratch, overwritten by the verification
 *                    pass), so hs_draft then also needs kv_len + k <= kv_capacity (HS_ERR_CAPACITY).
 * Whatever the plan, greedy verification emits the full model's own tokens (Sec. 3.3); the plan only moves the
 * acceptance rate and the cost of a draft step.  Synchronises; HS_ERR_ORDER between hs_draft and hs_verify. */
enum { HS_DRAFT_SKIP = 0, HS_DRAFT_LINEAR = 1, HS_DRAFT_FULL = 2 };
int hs_set_draft_plan(hs_model *m, const int32_t *plan_host);

/* Speculative sampling at temperature > 0 (paper Sec. 3.3, Eq. 6).  temperature = 0 (the default) is greedy decoding.
 * With temperature > 0: hs_draft draws draft i from softmax(draft logits / temperature) by inverse CDF with the uniform
 * u_draft_dev[b * max_k + i - 1] and keeps the draft logits; hs_accept_rollback (when no forced accept length is given)
 * accepts draft i iff u_accept_dev[b * max_k + i - 1] < P_H(x_i) / P_S(x_i), draws the correction at the first
 * rejection from the normalised positive part of P_H - P_S, or the bonus token after k acceptances from P_H, both with
 * u_final_dev[b]; the emitted tokens are then distributed as the full model's own samples.  The three DEVICE float
 * arrays ([max_batch][max_k], [max_batch][max_k], [max_batch], values in [0,1)) are read by the kernels of every
 * following round: the caller refills them between rounds (stream-ordered) and keeps them alive.  An inverse-CDF draw
 * takes the smallest index whose cumulative weight exceeds u * total.  Synchronises; HS_ERR_ORDER inside a round. */
int hs_set_sampling(hs_model *m, float temperature, const float *u_draft_dev, const float *u_accept_dev, const float *u_final_dev);

/* Verification phase (paper Sec. 3.3, "Verification phase": M_H, Eq. 2 / Eq. 3, processes the prefix and the
 * drafts in a single forward pass; here incrementally from the cached state) over k+1 candidates per sequence
 * at positions kv_len[b]..kv_len[b]+k.  k is passed explicitly so that k = 0 (plain autoregressive decoding,
 * the denominator of Eq. 1) and caller-supplied candidates need no preceding draft.
 * cand_dev: NULL to verify the candidates of the preceding hs_draft(k) (HS_ERR_ORDER if there was
 * none with this k, except k = 0), or int32 [batch][k+1] candidates to verify instead (cand[b][0]
 * replaces the pending token).  Produces g[b][i] = argmax of the logits after candidate i
 * (lowest id on ties), the top-2 margin, state snapshots and KV rows.  Ids in cand_dev outside [0, V) are
 * not used as addresses: token 0 is read instead and the device status word becomes HS_ERR_DEVICE.  Async.
 * HS_ERR_CAPACITY if a sequence could exceed kv_capacity; HS_ERR_ORDER if the previous hs_verify has not been
 * followed by hs_accept_rollback (its snapshots still hold the verified positions). */
int hs_verify(hs_model *m, int k, const int32_t *cand_dev);

/* Greedy acceptance + rollback after hs_verify (paper Sec. 3.3: under greedy decoding draft i is accepted iff
 * argmax P_S = argmax P_H at position i, and all tokens up to the first rejection are accepted; Eq. 1's
 * numerator counts the k+1 tokens a fully accepted round emits).  Per sequence: n = number of leading drafts with
 * cand[i+1] == g[i]; emitted = cand[1..n], g[n]; committed state <- snapshot n; kv_len += n+1;
 * pending <- g[n].  forced_n_dev (int32 [batch] on the device, or NULL) overrides n (0 <= n <= k) with
 * everything else unchanged; forced_next_dev (int32 [batch], entries < 0 ignored, or NULL) overrides
 * the next pending token.  n_acc_host [batch] / emitted_host [batch][k+1] (unused slots -1): if
 * either is non-NULL the results are copied to HOST memory and the stream is synchronised. */
int hs_accept_rollback(hs_model *m, const int32_t *forced_n_dev, const int32_t *forced_next_dev,
                       int32_t *n_acc_host, int32_t *emitted_host);

/* One whole round of paper Sec. 3.3 with HOST buffers: uploads forced_n_host / forced_next_host (either may be
 * NULL), runs draft(k), verify(k), accept/rollback, downloads n_acc_host [batch] and emitted_host [batch][k+1]
 * (either may be NULL) and synchronises.  HS_ERR_INVALID_ARG (nothing enqueued) if a forced accept length is
 * outside [0, k] or a forced next token is >= V. */
int hs_round_host(hs_model *m, int k, const int32_t *forced_n_host, const int32_t *forced_next_host,
                  int32_t *n_acc_host, int32_t *emitted_host);

/* ---- test and injection hooks (synchronous, host buffers) ---- */
enum { HS_STATE_SSM = 0,   /* f32 [H][P][N] committed Mamba-2 state of (layer, seq) */
       HS_STATE_CONV = 1,  /* f32 [3][channels] committed conv window (oldest row first) */
       HS_STATE_GDN = 2,   /* f32 [gh][gdv][gdk] committed DeltaNet state */
       HS_STATE_K = 3,     /* bf16 [rows][kvh][hd], rows = bytes / (kvh*hd*2), from row 0 */
       HS_STATE_V = 4,
       HS_STATE_DRAFT = 5, /* f32 draft scratch state after the last hs_draft; with HS_FLAG_LITERAL_DRAFT the draft
                              model's own committed state (export only) */
       HS_STATE_DRAFT_CONV = 6 /* f32 [3][channels] the draft model's own committed conv window (HS_FLAG_LITERAL_DRAFT; export only) */ };
int hs_export_state(hs_model *m, int layer, int seq, int kind, void *host, int64_t bytes);
int hs_import_state(hs_model *m, int layer, int seq, int kind, const void *host, int64_t bytes);
/* Declare sequence `seq` to hold kv_len consumed tokens and the given pending token (after imports);
 * batch = number of sequences that take part in the following rounds. */
int hs_set_context(hs_model *m, int seq, int kv_len, int pending);
int hs_set_batch(hs_model *m, int batch);
int hs_get_context(hs_model *m, int seq, int32_t *kv_len, int32_t *pending);
/* Logits [rows][V] f32 of the last pass (verify: row b*(k+1)+i; draft: last step, row b). */
int hs_get_logits(hs_model *m, float *host, int rows);
/* cand / g int32 [batch][k+1] and margin f32 [batch][k+1] of the last verify (any may be NULL). */
int hs_get_round(hs_model *m, int32_t *cand_host, int32_t *g_host, float *margin_host);
/* Number of kernels the library has launched (including those replayed inside graphs) so far. */
int64_t hs_launch_count(const hs_model *m);
/* Tuning hook for verify-mode attention (Sec. 3.3 verification pass): fix the split of the KV cache over
 * CTAs to `tiles` tiles of `chunk` keys per CTA for all following verify passes; chunk = 0 restores the
 * automatic choice (made per launch from the batch and the context lengths).  chunk is a multiple of 16 up to 128,
 * tiles 1..32, and chunk * tiles must be at least the chunk the workspace was laid out for (128, or less
 * for small batch * capacity): otherwise HS_ERR_INVALID_ARG and nothing changes.  A negative `tiles` with chunk = 128
 * selects the streaming form (-tiles tiles of 128 keys per CTA, partials merged by the last CTA to arrive) wherever the
 * attention runs as a launch of its own; it needs (qh / kvh) * (max_k + 1) <= 32.  Results do not depend on the setting
 * beyond fp32 summation order. */
int hs_set_attn_geometry(hs_model *m, int chunk, int tiles);
/* Tuning / measurement hook: switch a kernel choice on (value != 0) or off.  The choices are process-wide (they
 * apply to every handle); the handle's captured graphs are dropped so that the next step is captured afresh.
 * Results are the same within fp32 summation order.  Synchronises the stream.
 *   HS_OPT_CLUSTER_REDUCE  residual projections with 4..16 activation rows add the partial sums of their K split
 *                          inside a thread-block cluster (default on; off: the consumers add the parts)
 *   HS_OPT_GEMM_MMA        4..16 activation rows below the tcgen05 threshold on the warp-level tensor path (default on;
 *                          off: CUDA cores)
 *   HS_OPT_GEMM_TC         projections from HS_OPT_TC_MIN_ROWS activation rows on run on tcgen05 (default on; off: the
 *                          warp-level path, more than 16 rows as several 16-row launches)
 *   HS_OPT_PDL             programmatic dependent launch between the kernels of a pass (default on)
 *   HS_OPT_ATTN_SMALL      verify attention with at most 16 query rows per KV head over caches of up to 1024 keys
 *                          (2048 in a sequential hybrid) in its latency-lean form (default on; off: the general form)
 *   HS_OPT_ATTN_STREAM     verify attention over long caches at large batch (a launch of its own, at most 32 query rows
 *                          per KV head) in its streaming form (default on; off: the general form)
 *   HS_OPT_TC_MIN_ROWS     not a switch: the smallest number of activation rows (2..17) whose projections run on
 *                          tcgen05; 0 restores the automatic choice (7; 4 for models whose weight matrices are large
 *                          enough that the kernel's fixed cost is small beside the time to stream them) */
enum { HS_OPT_CLUSTER_REDUCE = 0, HS_OPT_GEMM_MMA = 1, HS_OPT_GEMM_TC = 2, HS_OPT_PDL = 3, HS_OPT_ATTN_SMALL = 4, HS_OPT_ATTN_STREAM = 5,
       HS_OPT_TC_MIN_ROWS = 6 };
int hs_set_option(hs_model *m, int option, int value);
/* Measurement hook.  hs_profile(m, 1) brackets every following kernel launch with two CUDA events on
 * the launching stream (graph replay is bypassed while it is on); hs_profile_read synchronises and
 * returns, per category, the summed device time in ms, the number of launches and the algorithmic
 * bytes the library attributes to them (projections: weights once + activations in + outputs;
 * 0 for the other categories).  Arrays have HS_PROF_COUNT entries.  hs_profile(m, 0) switches it
 * off and drops the records. */
enum { HS_PROF_GEMV = 0, HS_PROF_MIXER, HS_PROF_ATTN, HS_PROF_ARGMAX, HS_PROF_EMBED, HS_PROF_ACCEPT, HS_PROF_COUNT };
int hs_profile(hs_model *m, int enable);
int hs_profile_read(hs_model *m, double *ms, int64_t *launches, double *bytes);
/* Device status word: 0, or the first hs_status a kernel recorded.  Synchronises. */
int hs_device_status(hs_model *m);
/* Puts the status word back to 0 (async, on the model's stream). */
int hs_clear_status(hs_model *m);
/* Self-test of the bounded device-side wait: enqueues a one-warp kernel that waits `polls` (1..2^20) times on an
 * mbarrier nothing will ever complete, gives up and records HS_ERR_TIMEOUT, which hs_device_status then returns.
 * The kernel ends by itself; the handle stays usable (hs_clear_status).  Async. */
int hs_selftest_wait_timeout(hs_model *m, int polls);
/* Self-test of the kernels' own range checks: overwrites ONE device control word of sequence `seq` without the
 * validation every other entry point applies - HS_CTRL_KV_LEN (the cache length the attention kernels start from) or
 * HS_CTRL_SLOT (the index of the committed state snapshot the mixers start from).  Every kernel that turns such a
 * word into an address checks it first (cache length within [0, kv_capacity - rows], slot within the snapshot ring):
 * a block that finds it out of range touches neither the cache nor the state, and the status word becomes
 * HS_ERR_CAPACITY (cache too long) or HS_ERR_DEVICE.  The round's results are then meaningless; hs_reset or
 * hs_set_context + hs_import_state restore a consistent sequence, hs_clear_status the status word.  The host-side bounds
 * are not updated.  Synchronises.  HS_ERR_INVALID_ARG for a bad handle, sequence or word. */
enum { HS_CTRL_KV_LEN = 0, HS_CTRL_SLOT = 1 };
int hs_poke_control(hs_model *m, int seq, int word, int32_t value);
const char *hs_last_error(const hs_model *m);

/* Greedy argmax for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a convenience of the library.)  Computes, for each of `rows` logits rows of V floats (DEVICE,
 * row-major, contiguous), the id of the largest logit - the lowest id on a tie - into token_dev[row]
 * (DEVICE int32) and, if margin_dev is not NULL, top1 - top2 into margin_dev[row] (DEVICE float): the
 * same kernel and the same decisions as inside hs_draft / hs_verify.
 * Who needs it: code that may not call cudaMalloc where it runs - an engine that has already reserved
 * the whole GPU for its own pool, a component that is handed pointers and nothing else, a loop that
 * cannot afford the device-wide synchronisation an allocation can cause.  The kernel's scratch
 * (per-block partial results and arrival counters, 33 KB) therefore lives in a fixed __device__ array
 * inside the library; every GPU that loads libhs.so holds those 33 KB until the process ends.
 * Limits and rules:
 *  - rows <= 64, otherwise HS_ERR_SIZE and nothing is launched; V >= 1.  Bad pointers/sizes:
 *    HS_ERR_INVALID_ARG - that includes alignment: logits_dev must be 16-byte aligned when V is a multiple of 4
 *    (rows are then read 128 bits at a time; a view that starts inside a larger tensor may not be), 4-byte
 *    aligned otherwise, token_dev and margin_dev 4-byte aligned.  A failing CUDA call: HS_ERR_CUDA.
 *  - A row whose values are all -inf or NaN gets token 0 and margin 0.
 *  - The call allocates and frees nothing.  It is asynchronous on `stream` (a cudaStream_t).
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress) with
 *    that device current; make that first call outside any stream capture.
 *  - All calls share the one array: the counters are cleared at the start of every call, and two calls
 *    that may overlap on the GPU (different streams, no ordering between them) race on it - order them. */
int hs_argmax_static(const float *logits_dev, int V, int rows, int32_t *token_dev, float *margin_dev, void *stream);
int hs_destroy(hs_model *m);

#ifdef __cplusplus
}
#endif
#endif

// Internal declarations shared by the translation units of libhs (host orchestration + kernels).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string>
#include <vector>
#include <map>
#include "../../include/hs.h"

#define HS_MAX_K 8
#define HS_MAX_T (HS_MAX_K + 1)
#define HS_H_PARTS 4          // a projection may leave the residual stream as up to 4 partial sums
#define HS_ARGMAX_CHUNKS 32    // CTAs that share one logits row in the argmax
#define HS_MAX_GT 48          // (q heads per kv head) * (k+1) upper bound of the attention kernel

// ---------------------------------------------------------------------------------------------
// Control block in device memory (part of the caller's work buffer).  Everything a captured graph
// needs that changes from round to round lives here, so the graphs themselves never change.
// ---------------------------------------------------------------------------------------------
struct HsCtrl {
    int32_t *kv_len;      // [B]   consumed tokens per sequence
    int32_t *slot;        // [B]   snapshot index that holds the committed recurrent state
    int32_t *cand;        // [B][Tm] candidates of the current round; cand[b][0] = pending token
    int32_t *g;           // [B][Tm] full-model argmax after candidate i
    float *margin;        // [B][Tm] top1 - top2 of those logits
    int32_t *n_acc;       // [B]
    int32_t *emitted;     // [B][Tm]
    int32_t *stage_n;     // [B]   staging for host-supplied forced accept lengths
    int32_t *stage_next;  // [B]
    int32_t *status;      // [1]   first error a kernel recorded
    int32_t *counters;    // [B][kvh] split-KV arrival tickets (zero between launches)
    int32_t *am_counters; // [B][Tm] argmax arrival tickets (zero between launches)
    int32_t *dslot;       // [B]   slot of the draft model's own committed state (literal draft state)
};

struct HsLayer {
    int type;                 // HS_LAYER_*
    int rl;                   // ordinal among recurrent layers (PAR / GDN), else -1
    int al;                   // ordinal among layers with a KV cache (PAR / ATT), else -1
    const float *norm1, *conv_w, *conv_b, *A_log, *D, *dt_bias, *gnorm, *norm2;
    const __nv_bfloat16 *W_in, *W_out, *W_o, *W_gu, *W_down;
    int in_rows_full;         // rows of W_IN used in verify mode
    int in_rows_draft;        // rows used in draft mode (attention rows dropped)
};

struct hs_model {
    hs_config c;
    hs_buffers bufs;
    cudaStream_t stream;
    int B, Tm;                // max_batch, max_k + 1
    int nslot;                // state slots per (layer, sequence): Tm (snapshots) or 1 (rollback by replay)
    int log_w;                // floats of one logged update (replay mode), else 0
    float *ulog;              // [n_rl][B][Tm][log_w] update log (replay mode)
    int batch;                // active sequences
    int di, convd, gw;        // d_inner, conv channels, width of the gated mixer output
    int n_rl, n_al;           // recurrent layers, KV layers
    int64_t state_elems;      // floats of one (layer, seq) recurrent state
    int in_rows_max;
    int att_chunk, att_nch;   // keys per split, max splits
    int att_force_chunk, att_force_tiles;   // 0: automatic
    std::vector<HsLayer> layers;
    std::vector<int> plan;    // per-layer draft plan (HS_DRAFT_*)
    bool plan_attn;           // some layer of the draft runs attention (writes scratch KV rows beyond kv_len)
    const __nv_bfloat16 *embed, *lm_head;
    const float *final_norm;
    // carved out of bufs.work
    HsCtrl ctrl;
    float2 *rope;             // [cap][hd/2] (cos, sin)
    float *hbuf[2];            // residual stream, ping-pong; each [HS_H_PARTS][B*Tm][d] partial sums
    float *zx, *gbuf, *obuf, *abuf, *logits;
    float *dlogits;            // [B][max(max_k,1)][V] logits of the draft steps (kept for Eq. 6)
    float tau;                 // sampling temperature; 0: greedy
    const float *u_draft, *u_accept, *u_final;   // DEVICE uniforms of the round: [B][max_k], [B][max_k], [B]
    float *att_acc, *att_ml;
    __nv_bfloat16 *xb; int64_t xb_rows;   // packed activation operand of the many-row projection kernel
    std::vector<CUtensorMap> kmaps, vmaps;   // per attention layer (streaming attention form)
    int tc_min_rows_auto;                 // the automatic row threshold of the tcgen05 kernel for this model
    __nv_bfloat16 *xb_h, *xb_a; float *ssbuf;   // packed residual stream / MLP activations handed from projection to projection, row statistics
    void *am_part;             // argmax partials [B*Tm][HS_ARGMAX_CHUNKS] x 16 bytes
    // conv buffers
    float *cw, *hist, *dcw;
    float *dcwc, *dhist;       // literal draft state: the draft model's committed conv window and per-step raw inputs
    bool literal;              // the draft model keeps its own state over the whole history
    __nv_bfloat16 *Kc, *Vc;
    float *snap, *dstate;
    // host bookkeeping
    std::vector<int> kv_upper; // upper bound of kv_len per sequence (exact after a host readback)
    int phase;                 // 0 idle, 1 drafted, 2 verified
    int last_k;                // k of the last draft / verify
    bool sampled_draft;        // the draft logits buffer holds the distributions of the candidates now in `cand`
    int last_draft_k;          // draft length of the draft being enqueued (scratch KV rows of a plan that keeps attention)
    int last_rows;             // rows of logits of the last pass
    int64_t launches;
    std::string err;
    bool prof;                 // per-kernel event timing enabled
    struct ProfEvent { int cat; cudaEvent_t start, stop; double bytes; };
    std::vector<ProfEvent> prof_events;
    std::map<uint64_t, cudaGraphExec_t> graphs;
    std::map<uint64_t, int> graph_launches;
};

// ---------------------------------------------------------------------------------------------
// kernel launchers (each returns the cudaError_t of the launch)
// ---------------------------------------------------------------------------------------------
// Every kernel of a step is launched with programmatic stream serialization: it may start while its
// predecessor still runs and synchronises with griddepcontrol.wait (see hs_device.cuh).
extern bool g_hs_pdl;
extern bool g_hs_cluster_reduce; // residual projections of 4..16 rows reduce their K split inside a thread-block cluster
extern bool g_hs_gemm_mma;     // projections with 2..16 activation rows on the tensor cores (default) or the CUDA cores
// cluster_x > 1 launches thread-block clusters of that many CTAs along x (grid.x must be a multiple).
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                      int cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[2];
    int n = 0;
    if (cluster_x > 1) {
        at[n].id = cudaLaunchAttributeClusterDimension;
        at[n].val.clusterDim.x = cluster_x; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = 1;
        ++n;
    }
    if (g_hs_pdl) {
        at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = at; cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    return launch_pdl_cluster(kernel, grid, block, smem, s, 1, args...);
}
enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2 };

struct GemvArgs {
    // out[r][o] = sum_j W0[o][j] x0[r][j] (+ sum_j W1[o][j] x1[r][j]); x0 optionally RMS-normalised by norm_w.
    // x0 may be given as `xparts` partial sums (part p at x0 + p * xpstride), added in order.
    const __nv_bfloat16 *W0; int ldw0; int K0; const float *x0; int ldx0; int xparts; int64_t xpstride;
    const float *norm_w; float eps;
    const __nv_bfloat16 *W1; int ldw1; int K1; const float *x1; int ldx1;
    int O;                    // output rows of W (for SWIGLU: 2 * outputs)
    float *out; int ldo;      // [nrows][ldo]; EPI_RESID may write several parts, opstride floats apart
    int64_t opstride; int max_oparts;
    const float *resid; int rparts; int64_t rpstride;   // EPI_RESID: residual = sum of rparts parts, laid out like out
    int nrows;                // activation rows (batch * T), at most 16 per launch
    int epi;
    const void *pf_ptr; int64_t pf_bytes;   // optional: weights of the next projection, prefetched into L2
    __nv_bfloat16 *xb; int64_t xb_rows;     // scratch for the packed activation operand of the many-row kernel: [2][xb_rows][K0+K1]
    int early_trigger;        // 1: let the next kernel start before this one has waited for its predecessor
                              // (what a prologue may read before its own wait is stated in hs_device.cuh)
    // Many-row kernel only: projections hand the packed operand to each other, so that no packing kernel sits on the
    // dependent chain.  pk_in: the activations of this projection, already packed by the projection that produced them
    // ([2][rows per plane][K0], norm weight folded in, WITHOUT 1/rms when ss_in is given: ss_in[p * rows per plane + r],
    // p < ss_parts, are partial sums of squares of row r).  pk_out: where to leave this projection's result in packed
    // form for its consumer (row length pk_ld, times pk_nw[output] if given), with the partial sums of squares of the
    // residual epilogue's results in ss_out[128-row tile][rows per plane].
    const __nv_bfloat16 *pk_in; const float *ss_in; int ss_parts;
    __nv_bfloat16 *pk_out; int pk_ld; const float *pk_nw; float *ss_out;
};
// does a projection of nrows activation rows run on the many-row kernel?
bool gemv_uses_tc(int nrows, bool have_xb);
// *oparts receives the number of parts written to `out` (1 unless EPI_RESID split the reduction).
cudaError_t launch_gemv(const GemvArgs &a, int32_t *status, cudaStream_t s, int64_t *launches, int *oparts);
cudaError_t configure_gemv();   // one-time kernel attributes; call outside stream capture
// many activation rows (> 16): tcgen05 tensor-core contraction (kernels_gemm_tc.cu)
extern bool g_hs_gemm_tc;
extern int g_hs_tc_min_rows;      // projections with at least this many activation rows run on the tcgen05 kernel
cudaError_t configure_gemm_tc();
int gemm_tc_rows(int nrows);
cudaError_t launch_gemm_tc(const GemvArgs &a, int32_t *status, cudaStream_t s, int64_t *launches, int *oparts);
cudaError_t configure_attn();

// serial = true: launched in plain stream order (without the programmatic attribute); see model_pass
cudaError_t launch_embed(const __nv_bfloat16 *E, int d, int V, const int32_t *cand, int Tm, int col0, int T,
                         int b0, int nb, float *h, int32_t *status, bool serial, cudaStream_t s);

struct SsmArgs {
    int H, P, N, di, convd, in_ld;      // in_ld = row stride of zx
    const float *zx;                    // [rows][in_ld]: z | x B C | dt (| q k v)
    const float *conv_w, *conv_b, *A_log, *D, *dt_bias;
    const float *win_in;                // [B][3][convd] window the conv starts from
    float *win_out;                     // draft: [B][3][convd] shifted window; verify: NULL
    float *hist;                        // verify: [B][Tm][convd] raw inputs; draft: NULL
    const float *state_in;              // base of the state to read; per-seq stride + optional slot
    int64_t in_seq_stride, in_slot_stride;   // slot stride 0 => no slot indexing
    float *state_out;                   // verify: snapshots (slot i at i*out_slot_stride); draft: scratch
    int64_t out_seq_stride, out_slot_stride;
    const int32_t *slot;                // [B] committed slot (used when in_slot_stride != 0)
    // slot addressing: the state is read from slot (slot[b] + in_add) % slot_mod (slot_mod = 0: no wrap) and the state
    // after position i goes to slot i, or, with out_rel, to slot (slot[b] + out_add + i) % slot_mod
    int in_add, out_rel, out_add, slot_mod;
    float *g;                           // [rows][di] gated output y * silu(z)
    int T, Tm, b0, nb;
    float *log; int log_w;              // verify with rollback by replay: [B][Tm][log_w] update log (decay[H] | dt*x[di] | B[N]);
                                        // no state is stored.  NULL otherwise
    int nslot; int32_t *status;         // slot[b] must lie in [0, nslot): otherwise the block touches no state and
                                        // reports HS_ERR_DEVICE through the status word
};
cudaError_t launch_ssm(const SsmArgs &a, cudaStream_t s);

struct GdnArgs {
    int gh, dk, dv, convd, in_ld;
    const float *zx;                    // [rows][in_ld]: q | k | v | z | a | b
    const float *conv_w, *conv_b, *onorm; float eps;
    const float *win_in; float *win_out; float *hist;
    const float *state_in; int64_t in_seq_stride, in_slot_stride;
    float *state_out; int64_t out_seq_stride, out_slot_stride;
    const int32_t *slot;
    int in_add, out_rel, out_add, slot_mod;   // as in SsmArgs
    float *g;                           // [rows][gh*dv]
    int T, Tm, b0, nb;
    float *log; int log_w;              // rollback by replay: [B][Tm][log_w] (alpha[gh] | beta[gh] | k[gh*dk] | v[gh*dv]); NULL otherwise
    int nslot; int32_t *status;         // as in SsmArgs
};
cudaError_t launch_gdn(const GdnArgs &a, cudaStream_t s);

// Rollback by replay: apply the first n_acc[b] + 1 logged updates of every recurrent layer to the committed state in place.
struct ReplayArgs {
    int arch;                           // HS_ARCH_*
    int H, P, N, di;                    // Mamba-2
    int gh, dk, dv;                     // DeltaNet
    float *state;                       // [n_rl][B][state]
    const float *log; int log_w;        // [n_rl][B][Tm][log_w]
    const int32_t *n_acc;               // [B]; must lie in [0, Tm): otherwise nothing is applied and the status word reports it
    int64_t state_elems;
    int n_rl, B, Tm, b0, nb;
    int32_t *status;
};
cudaError_t launch_replay(const ReplayArgs &a, cudaStream_t s);

struct AttnArgs {
    int qh, kvh, hd, in_ld, q_off, k_off, v_off;
    const float *zx;
    const float2 *rope;                 // [cap][hd/2]
    __nv_bfloat16 *Kc, *Vc;             // this layer: [B][kvh][cap][hd]
    int cap;
    const int32_t *kv_len;
    float *o;                           // [rows][qh*hd]
    float *part_acc, *part_ml; int32_t *counters; int32_t *status;
    int chunk, tiles, nch;              // keys per tile, tiles per CTA, CTAs (key ranges) that cover the cache capacity
    int len_off;                        // the new rows start at kv_len[b] + len_off (draft step i of a plan that keeps attention: i)
    int stream;                         // 1: the streaming form for long caches (stand-alone launches: chunk = 128, at most 32 query rows)
    int small;                          // 1: the latency-lean form (G*T <= 16 rows, every cache within one cluster of 8 CTAs x chunk keys)
    int T, b0, nb;
    // streaming form: this layer's K and V cache as 2-D tensors [B * kvh * cap rows][hd] for tiled bulk copies
    // (boxes of 64 columns x 128 rows, 128-byte swizzle); made once per layer by hs_make_kv_tensor_map
    alignas(64) CUtensorMap kmap, vmap;
};
cudaError_t launch_attn(const AttnArgs &a, cudaStream_t s);
extern bool g_hs_tensor_maps;   // the driver's tensor-map encoder was found (configure_gemm_tc)
cudaError_t hs_make_kv_tensor_map(CUtensorMap *map, const void *base, uint64_t rows, int hd);
// mixer + attention of a parallel block in one launch (verify pass); *fused = false: not applicable, nothing launched
cudaError_t launch_ssm_attn(const SsmArgs &sa, const AttnArgs &a, cudaStream_t s, bool *fused);
bool ssm_wide(const SsmArgs &a);    // the mixer runs a whole head per block (large batch)

// part: scratch of HS_ARGMAX_CHUNKS * 16 bytes per logits row (row slot b * Tm + i); counters: one int32 per
// row slot, zero between launches
cudaError_t launch_argmax(const float *logits, int V, int T, int b0, int nb, int Tm,
                          int32_t *tok_out, int tok_col0, float *margin_out, void *part, int32_t *counters, cudaStream_t s);

struct AcceptArgs {
    int k, Tm, b0, nb, n_rl, B, convd, V, replay;   // replay: the committed state stays in slot 0
    HsCtrl ctrl;
    const int32_t *forced_n, *forced_next;
    float *cw; const float *hist;       // [n_rl][B][3][convd], [n_rl][B][Tm][convd]
    float *dcw; const float *dhist;     // the draft model's own committed window and raw inputs (literal draft state), or NULL
    int32_t *dslot; int dslot_mod;      // its committed slot advances by n + 1 (mod dslot_mod)
};
cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t s);
cudaError_t launch_wait_probe(int32_t *status, int polls, cudaStream_t s);
// speculative sampling (Eq. 6): a draft draw from softmax(logits / tau), and the accept / correction / bonus decision
cudaError_t launch_sample(const float *logits, int64_t row_stride, int V, int Tm, int b0, int nb, float tau,
                          const float *u, int u_stride, int u_col, int32_t *tok_out, int tok_col, cudaStream_t s);
cudaError_t launch_spec_accept(const float *dlogits, int64_t d_seq_stride, const float *vlogits, const int32_t *cand,
                               const float *u_acc, const float *u_final, int u_stride, int32_t *n_out, int32_t *next_out,
                               int V, int Tm, int k, int b0, int nb, float tau, cudaStream_t s);

// C-ABI of libhs: buffer layout, the fixed kernel sequence of a draft step and of a verify pass,
// CUDA-graph replay of those sequences, and the test / injection hooks.  See include/hs.h.
#include "hs_internal.h"
#include <cmath>
#include <cstdio>
#include <cstring>
#include <algorithm>

bool g_hs_attn_small = true;   // short caches and few query rows use the latency-lean attention form
bool g_hs_attn_stream = true;  // long caches at large batch use the streaming attention form

namespace {

constexpr int64_t ALIGN = 256;
inline int64_t up(int64_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

int layer_type(const hs_config &c, int l) {
    if (c.arch == HS_ARCH_PARALLEL) return HS_LAYER_PAR;
    return (l % 4 == 3) ? HS_LAYER_ATT : HS_LAYER_GDN;
}
int d_inner(const hs_config &c) { return c.H * c.P; }
int conv_channels(const hs_config &c) {
    return c.arch == HS_ARCH_PARALLEL ? c.H * c.P + 2 * c.N : 2 * c.gh * c.gdk + c.gh * c.gdv;
}
int attn_rows(const hs_config &c) { return (c.qh + 2 * c.kvh) * c.hd; }
int in_rows(const hs_config &c, int type, bool draft) {
    if (type == HS_LAYER_PAR) return 2 * d_inner(c) + 2 * c.N + c.H + (draft ? 0 : attn_rows(c));
    if (type == HS_LAYER_GDN) return 2 * c.gh * c.gdk + 2 * c.gh * c.gdv + 2 * c.gh;
    return attn_rows(c);
}

struct TensorDesc { int id; int64_t elems; int esize; };

int layer_tensors(const hs_config &c, int type, TensorDesc *out) {
    int n = 0;
    const int64_t d = c.d, di = d_inner(c), cd = conv_channels(c);
    out[n++] = {HS_T_NORM1, d, 4};
    out[n++] = {HS_T_W_IN, (int64_t)in_rows(c, type, false) * d, 2};
    if (type == HS_LAYER_PAR) {
        out[n++] = {HS_T_CONV_W, cd * 4, 4}; out[n++] = {HS_T_CONV_B, cd, 4};
        out[n++] = {HS_T_A_LOG, c.H, 4}; out[n++] = {HS_T_D, c.H, 4}; out[n++] = {HS_T_DT_BIAS, c.H, 4};
        out[n++] = {HS_T_GNORM, di, 4};
        out[n++] = {HS_T_W_OUT, d * di, 2}; out[n++] = {HS_T_W_O, d * c.qh * c.hd, 2};
    } else if (type == HS_LAYER_GDN) {
        out[n++] = {HS_T_CONV_W, cd * 4, 4}; out[n++] = {HS_T_CONV_B, cd, 4};
        out[n++] = {HS_T_GNORM, c.gdv, 4};
        out[n++] = {HS_T_W_OUT, d * c.gh * c.gdv, 2};
    } else {
        out[n++] = {HS_T_W_O, d * c.qh * c.hd, 2};
    }
    out[n++] = {HS_T_NORM2, d, 4};
    out[n++] = {HS_T_W_GU, (int64_t)2 * c.ff * d, 2};
    out[n++] = {HS_T_W_DOWN, d * c.ff, 2};
    return n;
}

// byte offset of (layer, tensor) in the blob, or the total size when layer == L
int64_t blob_offset(const hs_config &c, int layer, int tensor) {
    int64_t off = 0;
    const int64_t g[3] = {(int64_t)c.V * c.d * 2, (int64_t)c.V * c.d * 2, (int64_t)c.d * 4};
    for (int t = 0; t < 3; ++t) {
        if (layer == -1 && tensor == t) return off;
        off = up(off + g[t]);
    }
    if (layer == -1) return -1;
    TensorDesc td[HS_T_COUNT];
    for (int l = 0; l < c.L; ++l) {
        int n = layer_tensors(c, layer_type(c, l), td);
        for (int i = 0; i < n; ++i) {
            if (l == layer && td[i].id == tensor) return off;
            off = up(off + td[i].elems * td[i].esize);
        }
        if (l == layer) return -1;
    }
    return off;   // layer == L: total
}

bool valid_config(const hs_config &c) {
    if (c.L < 1 || c.d < 256 || (c.d & 255) || c.V < 2 || (c.ff & 255) || c.ff < 256) return false;
    if (c.conv_w != 4 || c.max_k < 0 || c.max_k > HS_MAX_K || c.max_batch < 1 || c.kv_capacity < 1) return false;
    if (c.hd != 64 && c.hd != 128) return false;
    if (c.qh < 1 || c.kvh < 1 || c.qh % c.kvh) return false;
    if ((c.qh / c.kvh) * (c.max_k + 1) > HS_MAX_GT) return false;
    if ((c.qh * c.hd) & 255) return false;
    if (c.arch == HS_ARCH_PARALLEL) {
        if (c.H < 1 || c.P < 16 || (c.P & 15)) return false;
        if (c.N != 64 && c.N != 128 && c.N != 256) return false;
        if ((c.H * c.P) & 255) return false;
        if ((2 * c.H * c.P + 2 * c.N + c.H) & 3) return false;   // attention rows must start 16-byte aligned
    } else if (c.arch == HS_ARCH_SEQUENTIAL) {
        if (c.gh < 1 || c.gdk != 64 || c.gdv < 16 || c.gdv > 64 || (c.gdv & 15)) return false;
        if ((c.gh * c.gdv) & 255) return false;
    } else return false;
    return true;
}

struct Derived {
    int B, Tm, R, n_rl, n_al, convd, gw, in_rows_max, att_chunk, att_nch;
    int nslot, log_w;         // state slots per (layer, sequence); floats of one logged update (rollback by replay)
    int literal;              // the draft model keeps its own state: a ring of Tm + 1 draft slots, a second set of conv buffers
    int64_t state_elems;
};

Derived derive(const hs_config &c) {
    Derived v;
    v.B = c.max_batch; v.Tm = c.max_k + 1; v.R = v.B * v.Tm;
    v.n_rl = v.n_al = 0; v.in_rows_max = 0;
    for (int l = 0; l < c.L; ++l) {
        int t = layer_type(c, l);
        if (t != HS_LAYER_ATT) ++v.n_rl;
        if (t != HS_LAYER_GDN) ++v.n_al;
        int r = in_rows(c, t, false);
        if (r > v.in_rows_max) v.in_rows_max = r;
    }
    v.convd = conv_channels(c);
    v.gw = c.arch == HS_ARCH_PARALLEL ? d_inner(c) : c.gh * c.gdv;
    v.state_elems = c.arch == HS_ARCH_PARALLEL ? (int64_t)c.H * c.P * c.N : (int64_t)c.gh * c.gdv * c.gdk;
    const bool replay = (c.flags & HS_FLAG_REPLAY) != 0;
    v.nslot = replay ? 1 : v.Tm;
    v.literal = (c.flags & HS_FLAG_LITERAL_DRAFT) ? 1 : 0;
    v.log_w = !replay ? 0 : c.arch == HS_ARCH_PARALLEL ? c.H + c.H * c.P + c.N : c.gh * (2 + c.gdk + c.gdv);
    // keys per attention CTA: the largest of 128 / 64 / 32 that still gives about two CTAs per SM
    int chunk = 128;
    while (chunk > 32 && (int64_t)c.max_batch * c.kvh * ((c.kv_capacity + chunk - 1) / chunk) < 296) chunk >>= 1;
    v.att_chunk = chunk;
    v.att_nch = (c.kv_capacity + chunk - 1) / chunk;
    return v;
}

// layout of the work buffer; base may be null to only measure
struct WorkLayout {
    int64_t kv_len, slot, cand, g, margin, n_acc, emitted, stage_n, stage_next, status, counters, am_counters, dslot;
    int64_t rope, h, zx, gbuf, obuf, abuf, logits, dlogits, att_acc, att_ml, am_part, xb, xb_h, xb_a, ssbuf, total;
};

WorkLayout work_layout(const hs_config &c, const Derived &v) {
    WorkLayout w; int64_t off = 0;
    auto take = [&](int64_t bytes) { int64_t o = off; off = up(off + bytes); return o; };
    w.kv_len = take(4 * v.B); w.slot = take(4 * v.B);
    w.cand = take(4 * v.R); w.g = take(4 * v.R); w.margin = take(4 * v.R);
    w.n_acc = take(4 * v.B); w.emitted = take(4 * v.R);
    w.stage_n = take(4 * v.B); w.stage_next = take(4 * v.B);
    w.status = take(4); w.counters = take((int64_t)4 * v.B * c.kvh); w.am_counters = take((int64_t)4 * v.R);
    w.dslot = take(4 * v.B);
    w.rope = take((int64_t)c.kv_capacity * (c.hd / 2) * 8);
    w.h = take((int64_t)4 * 2 * HS_H_PARTS * v.R * c.d);
    w.zx = take((int64_t)4 * v.R * v.in_rows_max);
    w.gbuf = take((int64_t)4 * v.R * v.gw);
    w.obuf = take((int64_t)4 * v.R * c.qh * c.hd);
    w.abuf = take((int64_t)4 * v.R * c.ff);
    w.logits = take((int64_t)4 * v.R * c.V);
    w.dlogits = take((int64_t)4 * v.B * std::max(c.max_k, 1) * c.V);
    w.att_acc = take((int64_t)4 * v.B * c.kvh * v.att_nch * HS_MAX_GT * c.hd);
    w.att_ml = take((int64_t)4 * v.B * c.kvh * v.att_nch * HS_MAX_GT * 2);
    w.am_part = take((int64_t)16 * v.R * HS_ARGMAX_CHUNKS);
    {   // packed bf16 activation operand of the many-row projection kernel: [2][rows][widest reduction]
        const int64_t kmax = std::max<int64_t>(std::max<int64_t>(c.d, c.ff), (int64_t)v.gw + c.qh * c.hd);
        const int64_t pr = gemm_tc_rows(v.R);
        w.xb = take((int64_t)2 * 2 * pr * kmax);
        // the same for the residual stream and the MLP activations, written by the producing projection's epilogue,
        // and the partial sums of squares (one per 128 model dimensions) of the residual stream's rows
        w.xb_h = take((int64_t)2 * 2 * pr * c.d);
        w.xb_a = take((int64_t)2 * 2 * pr * c.ff);
        w.ssbuf = take((int64_t)4 * pr * ((c.d + 127) / 128));
    }
    w.total = off;
    return w;
}

int fail(hs_model *m, int code, const char *msg) {
    if (m) m->err = msg;
    return code;
}
int cuda_fail(hs_model *m, cudaError_t e, const char *where) {
    if (m) { m->err = std::string(where) + ": " + cudaGetErrorString(e); }
    return HS_ERR_CUDA;
}
#define CK(call, where) do { cudaError_t e__ = (call); if (e__ != cudaSuccess) return cuda_fail(m, e__, where); } while (0)

// Per-kernel timing (measurement hook): when enabled, every launch is bracketed by two events on the
// launching stream; hs_profile_read sums the elapsed times per category.
void prof_mark(hs_model *m, int cat, bool begin, double bytes) {
    if (!m->prof) return;
    cudaEvent_t ev;
    if (cudaEventCreate(&ev) != cudaSuccess) return;
    cudaEventRecord(ev, m->stream);
    if (begin) m->prof_events.push_back({cat, ev, nullptr, 0.0});
    else { m->prof_events.back().stop = ev; m->prof_events.back().bytes = bytes; }
}
#define PROF(cat, bytes, call, where) do { prof_mark(m, cat, true, 0); CK(call, where); prof_mark(m, cat, false, bytes); } while (0)

double gemv_bytes(const GemvArgs &a) {
    // weights once (bf16) + activation rows in (fp32) + outputs (fp32; residual read as well)
    const double Kt = (double)a.K0 + a.K1, outs = a.epi == EPI_SWIGLU ? a.O / 2 : a.O;
    return (double)a.O * Kt * 2 + (double)a.nrows * Kt * 4 + (double)a.nrows * outs * 4 * (a.epi == EPI_RESID ? 2 : 1);
}

// ------------------------------------------------------------------------------------------------
// one pass of the model over T positions per sequence (sequences b0 .. b0+nb-1)
//   draft = false: full model M_H (verify);  draft = true: draft model M_S, one position,
//   reading candidate column `col` and, for step > 0, the scratch state of the previous step.
// ------------------------------------------------------------------------------------------------
// Attention geometry of this launch.  Keys per tile: the context is spread over the eight CTAs of one
// cluster (which combine their partials in shared memory) - 32, 64, 96 or 128 keys each, whichever first
// covers it - and never below the size the partial buffers were laid out for; longer contexts use 128-key
// tiles over several clusters.  Tiles per CTA: one, unless the launch would have far more CTAs than the GPU
// runs at once (long caches at large batch) - then a CTA walks up to sixteen 64-key tiles, so that staging
// the queries and combining the partials is paid once per 1024 keys.
// Few query rows (G * T <= 16) over caches that fit one cluster: the latency-lean attention form, keys per CTA in
// steps of 32 up to 128 (parallel blocks: the mixer CTAs of the fused launch get the same shared memory) or 256.
struct AttnGeom {
    int chunk, tiles, small, stream;
    int code() const { return stream * 1024 + small * 512 + (chunk / 16 - 1) * 32 + tiles - 1; }   // < 2048, part of the graph key
};
// Tq: query positions per sequence of the launch; T: rows the pass may append beyond the upper bound of kv_len
// (the same for a verify pass; a draft that keeps attention appends one row per step, k in all)
AttnGeom attn_geom(const hs_model *m, int Tq, int T, int b0, int nb) {
    if (m->att_force_chunk) return AttnGeom{m->att_force_chunk, m->att_force_tiles < 0 ? -m->att_force_tiles : m->att_force_tiles, 0, m->att_force_tiles < 0 ? 1 : 0};
    const bool have_maps = !m->kmaps.empty();        // the streaming form fetches its tiles with tensor copies
    int maxlen = 0;
    for (int b = b0; b < b0 + nb; ++b) if (m->kv_upper[b] > maxlen) maxlen = m->kv_upper[b];
    {
        const int limit = m->c.arch == HS_ARCH_PARALLEL ? 128 : 256;
        int ck = 32;
        while (ck < limit && 8 * ck < maxlen + T) ck += 32;
        if (g_hs_attn_small && (m->c.qh / m->c.kvh) * Tq <= 16 && 8 * ck >= maxlen + T) return AttnGeom{ck, 1, 1, 0};
    }
    int want = 32;
    while (want < 128 && 8 * want < maxlen + T) want += 32;
    // Long caches at a batch that fills the GPU several times over, in a launch of its own (not fused with the mixer):
    // the streaming form - 128-key tiles, up to 16 per CTA.
    {
        const bool own_launch = m->c.arch == HS_ARCH_SEQUENTIAL || (int64_t)(m->c.P / 16) * m->c.H * nb > 4 * 148;
        const int64_t ctas128 = (int64_t)nb * m->c.kvh * ((maxlen + T + 127) / 128);
        if (g_hs_attn_stream && have_maps && own_launch && (m->c.qh / m->c.kvh) * Tq <= 32 && ctas128 >= 2 * 148) {
            // tiles per CTA: up to 16, fewer only while that still leaves about half an SM count of CTAs (measured: 544 tiles
            // of work run best as 8 per CTA - staging the queries and merging the ranges is paid per CTA)
            int tiles = (int)((ctas128 + 73) / 74);
            tiles = tiles < 1 ? 1 : tiles > 16 ? 16 : tiles;
            return AttnGeom{128, tiles, 0, 1};
        }
    }
    AttnGeom g{want > m->att_chunk ? want : m->att_chunk, 1, 0, 0};
    const int64_t ctas64 = (int64_t)nb * m->c.kvh * ((maxlen + T + 63) / 64);
    const int64_t fill = 148 * 8;             // CTAs that keep every SM busy for several rounds
    if (g.chunk == 128 && ctas64 >= 4 * fill) {
        g.chunk = 64;
        g.tiles = ctas64 / fill >= 16 ? 16 : ctas64 / fill >= 8 ? 8 : ctas64 / fill >= 4 ? 4 : 2;
    } else if (g.chunk == 128 && maxlen + T > 8 * 128) {
        // a cache beyond one cluster of 128-key ranges: as many tiles per CTA as keep it inside ONE cluster, which spares
        // the merge of several clusters' partials through global memory (measured, 2048 keys: 2-3 % per verify pass)
        int t = (maxlen + T + 8 * 128 - 1) / (8 * 128);
        t = t < 4 ? (t < 2 ? 2 : 4) : t;              // measured: four tiles beat two and three at 2048 keys
        g.tiles = t > 16 ? 16 : t;
    }
    return g;
}

// does the draft run layer l at all?  (a skipped layer and an attention layer that is not kept whole are the identity)
inline bool draft_runs(const hs_model *m, int l) {
    return m->plan[l] != HS_DRAFT_SKIP && (m->layers[l].type != HS_LAYER_ATT || m->plan[l] == HS_DRAFT_FULL);
}

// first = true: this pass opens an API call (its predecessor in the stream may be the accept kernel of the last
// round): its first kernel goes out in plain stream order, see hs_device.cuh.
// chunk = true (literal draft state only): the DRAFT model over T positions of every sequence on its own state buffers,
// like a verify pass of M_S (prompt chunks; candidates supplied by the caller); head = false: no LM head / token choice.
int model_pass(hs_model *m, bool draft, int T, int step, int b0, int nb, bool first, bool chunk = false, bool head = true) {
    const hs_config &c = m->c;
    const AttnGeom at_geom = draft ? attn_geom(m, 1, m->last_draft_k, b0, nb) : attn_geom(m, T, T, b0, nb);
    cudaStream_t s = m->stream;
    const int rows = nb * T, d = c.d;
    const int64_t se = m->state_elems;
    // the residual stream ping-pongs between two buffers; a projection that splits its reduction
    // leaves it as `hparts` partial sums, which every consumer adds in order
    int cur = 0, hparts = 1;
    const int64_t hps = (int64_t)m->B * m->Tm * d;
    int32_t *st_w = m->ctrl.status;
    // many rows: every projection of the pass runs on the tcgen05 kernel, and the projections hand each other their
    // results in the packed form that kernel consumes (only the mixer's output and the embedding are packed by a
    // kernel of their own)
    const bool tc_pass = gemv_uses_tc(rows, m->xb != nullptr);
    const int ss_parts = (d + 127) / 128;
    bool h_packed = false;                  // xb_h / ssbuf hold the current residual stream
    PROF(HS_PROF_EMBED, 0, launch_embed(m->embed, d, c.V, m->ctrl.cand, m->Tm, draft ? step : 0, T, b0, nb, m->hbuf[0], st_w, first, s), "embed");
    ++m->launches;
    for (int l = 0; l < c.L; ++l) {
        const HsLayer &ly = m->layers[l];
        // the full model runs every layer whole; the draft follows its per-layer plan (default: the recurrent pathway of
        // every layer - Eq. 4 - which makes an attention layer of a sequential hybrid the identity - Eq. 5)
        if (draft && !draft_runs(m, l)) continue;
        const bool with_attn = ly.type != HS_LAYER_GDN && (!draft || m->plan[l] == HS_DRAFT_FULL);
        const int inr = with_attn ? ly.in_rows_full : ly.in_rows_draft;
        // (1) RMSNorm + in-projection (verify: Mamba rows and q|k|v rows in one pass over u)
        GemvArgs ga{};
        ga.W0 = ly.W_in; ga.ldw0 = d; ga.K0 = d; ga.x0 = m->hbuf[cur]; ga.ldx0 = d; ga.xparts = hparts; ga.xpstride = hps;
        ga.norm_w = ly.norm1; ga.eps = c.eps;
        ga.O = inr; ga.out = m->zx; ga.ldo = m->in_rows_max; ga.nrows = rows; ga.epi = EPI_STORE;
        ga.early_trigger = 1;
        ga.pf_ptr = ly.type == HS_LAYER_ATT ? ly.W_o : ly.W_out;
        ga.pf_bytes = 2 * (int64_t)d * (ly.type == HS_LAYER_ATT ? c.qh * c.hd : m->gw);
        ga.xb = m->xb; ga.xb_rows = m->xb_rows;
        if (tc_pass && h_packed) { ga.pk_in = m->xb_h; ga.ss_in = m->ssbuf; ga.ss_parts = ss_parts; }
        PROF(HS_PROF_GEMV, gemv_bytes(ga), launch_gemv(ga, st_w, s, &m->launches, nullptr), "in_proj");
        // (2) recurrent mixer
        SsmArgs ssm_args{};
        bool ssm_deferred = false;
        if (ly.type != HS_LAYER_ATT) {
            const size_t lrB = (size_t)ly.rl * m->B;
            const float *win_in; float *win_out = nullptr, *hist = nullptr;
            const size_t half = (size_t)m->n_rl * m->B * 3 * m->convd;
            const bool lit = draft && m->literal;          // the draft model runs on its own state buffers
            if (!draft) { win_in = m->cw + lrB * 3 * m->convd; hist = m->hist + lrB * m->Tm * m->convd; }
            else if (chunk) { win_in = m->dcwc + lrB * 3 * m->convd; hist = m->dhist + lrB * m->Tm * m->convd; }
            else {
                const float *committed = lit ? m->dcwc : m->cw;
                win_in = step == 0 ? committed + lrB * 3 * m->convd : m->dcw + ((step - 1) & 1) * half + lrB * 3 * m->convd;
                win_out = m->dcw + (step & 1) * half + lrB * 3 * m->convd;
                if (lit) hist = m->dhist + lrB * m->Tm * m->convd + (size_t)step * m->convd;     // raw inputs of draft position `step`
            }
            const float *st_in; int64_t in_seq, in_slot; float *st_out; int64_t out_seq, out_slot;
            const int32_t *slot_arr = m->ctrl.slot;
            int in_add = 0, out_rel = 0, out_add = 0, slot_mod = 0;
            // snapshots: slot i of (layer, sequence) holds the state after position i and `slot` names the committed one;
            // rollback by replay: one slot, the committed state, and the verify pass writes the update log instead
            const int64_t ns = m->nslot;
            const bool replay = m->log_w != 0;
            float *snap_l = m->snap + lrB * ns * se, *dst_l = m->dstate + lrB * se;
            float *log_l = (!draft && replay) ? m->ulog + lrB * m->Tm * m->log_w : nullptr;
            if (!draft) { st_in = snap_l; in_seq = ns * se; in_slot = replay ? 0 : se; st_out = snap_l; out_seq = ns * se; out_slot = replay ? 0 : se; }
            else if (lit) {
                // literal draft state: a ring of Tm + 1 slots per (layer, sequence); the committed slot dslot[b] is never
                // overwritten during a round: draft position i reads slot dslot + i and writes slot dslot + i + 1
                const int64_t dn = m->Tm + 1;
                float *ring = m->dstate + lrB * dn * se;
                st_in = ring; in_seq = dn * se; in_slot = se; st_out = ring; out_seq = dn * se; out_slot = se;
                slot_arr = m->ctrl.dslot; slot_mod = (int)dn; out_rel = 1;
                in_add = chunk ? 0 : step; out_add = chunk ? 1 : step + 1;
            }
            else if (step == 0) { st_in = snap_l; in_seq = ns * se; in_slot = replay ? 0 : se; st_out = dst_l; out_seq = se; out_slot = 0; }
            else { st_in = dst_l; in_seq = se; in_slot = 0; st_out = dst_l; out_seq = se; out_slot = 0; }
            if (ly.type == HS_LAYER_PAR) {
                SsmArgs sa{};
                sa.H = c.H; sa.P = c.P; sa.N = c.N; sa.di = m->di; sa.convd = m->convd; sa.in_ld = m->in_rows_max;
                sa.zx = m->zx; sa.conv_w = ly.conv_w; sa.conv_b = ly.conv_b; sa.A_log = ly.A_log; sa.D = ly.D; sa.dt_bias = ly.dt_bias;
                sa.win_in = win_in; sa.win_out = win_out; sa.hist = hist;
                sa.state_in = st_in; sa.in_seq_stride = in_seq; sa.in_slot_stride = in_slot;
                sa.state_out = st_out; sa.out_seq_stride = out_seq; sa.out_slot_stride = out_slot;
                sa.slot = slot_arr; sa.in_add = in_add; sa.out_rel = out_rel; sa.out_add = out_add; sa.slot_mod = slot_mod; sa.g = m->gbuf; sa.T = T; sa.Tm = m->Tm; sa.b0 = b0; sa.nb = nb;
                sa.log = log_l; sa.log_w = m->log_w;
                sa.nslot = slot_mod ? slot_mod : (int)ns; sa.status = st_w;
                if (with_attn) { ssm_args = sa; ssm_deferred = true; }      // goes out together with the attention
                else PROF(HS_PROF_MIXER, 0, launch_ssm(sa, s), "ssm");
            } else {
                GdnArgs gd{};
                gd.gh = c.gh; gd.dk = c.gdk; gd.dv = c.gdv; gd.convd = m->convd; gd.in_ld = m->in_rows_max;
                gd.zx = m->zx; gd.conv_w = ly.conv_w; gd.conv_b = ly.conv_b; gd.onorm = ly.gnorm; gd.eps = c.eps;
                gd.win_in = win_in; gd.win_out = win_out; gd.hist = hist;
                gd.state_in = st_in; gd.in_seq_stride = in_seq; gd.in_slot_stride = in_slot;
                gd.state_out = st_out; gd.out_seq_stride = out_seq; gd.out_slot_stride = out_slot;
                gd.slot = slot_arr; gd.in_add = in_add; gd.out_rel = out_rel; gd.out_add = out_add; gd.slot_mod = slot_mod; gd.g = m->gbuf; gd.T = T; gd.Tm = m->Tm; gd.b0 = b0; gd.nb = nb;
                gd.log = log_l; gd.log_w = m->log_w;
                gd.nslot = slot_mod ? slot_mod : (int)ns; gd.status = st_w;
                PROF(HS_PROF_MIXER, 0, launch_gdn(gd, s), "gdn");
            }
            if (!ssm_deferred) ++m->launches;
        }
        // (3) attention over the cache + the new rows (full model only)
        if (with_attn) {
            AttnArgs aa{};
            aa.qh = c.qh; aa.kvh = c.kvh; aa.hd = c.hd; aa.in_ld = m->in_rows_max;
            aa.q_off = ly.type == HS_LAYER_PAR ? ly.in_rows_draft : 0;
            aa.k_off = aa.q_off + c.qh * c.hd; aa.v_off = aa.k_off + c.kvh * c.hd;
            aa.zx = m->zx; aa.rope = m->rope;
            const size_t per_layer = (size_t)m->B * c.kvh * c.kv_capacity * c.hd;
            aa.Kc = m->Kc + ly.al * per_layer; aa.Vc = m->Vc + ly.al * per_layer; aa.cap = c.kv_capacity;
            aa.kv_len = m->ctrl.kv_len; aa.o = m->obuf;
            aa.part_acc = m->att_acc; aa.part_ml = m->att_ml; aa.counters = m->ctrl.counters; aa.status = m->ctrl.status;
            aa.chunk = at_geom.chunk; aa.tiles = at_geom.tiles; aa.small = at_geom.small; aa.stream = at_geom.stream;
            if (!m->kmaps.empty()) { aa.kmap = m->kmaps[ly.al]; aa.vmap = m->vmaps[ly.al]; }
            aa.len_off = draft ? step : 0;
            aa.nch = (c.kv_capacity + at_geom.chunk * at_geom.tiles - 1) / (at_geom.chunk * at_geom.tiles); aa.T = T; aa.b0 = b0; aa.nb = nb;
            bool fused = false;
            if (ssm_deferred) {
                // a parallel block: mixer and attention are independent of each other - one launch for both
                if (!ssm_wide(ssm_args)) PROF(HS_PROF_MIXER, 0, launch_ssm_attn(ssm_args, aa, s, &fused), "ssm + attention");
                if (fused) ++m->launches;
                else { PROF(HS_PROF_MIXER, 0, launch_ssm(ssm_args, s), "ssm"); ++m->launches; }
            }
            if (!fused) {
                PROF(HS_PROF_ATTN, 0, launch_attn(aa, s), "attention");
                ++m->launches;
            }
        }
        // (4) out-projection(s) + residual:  h += W_out rmsnorm_gated(g)  (+ W_o o)
        GemvArgs go{};
        go.O = d; go.out = m->hbuf[cur ^ 1]; go.ldo = d; go.opstride = hps; go.max_oparts = HS_H_PARTS;
        go.resid = m->hbuf[cur]; go.rparts = hparts; go.rpstride = hps; go.nrows = rows; go.epi = EPI_RESID; go.xparts = 1;
        if (ly.type == HS_LAYER_PAR) {
            go.W0 = ly.W_out; go.ldw0 = m->di; go.K0 = m->di; go.x0 = m->gbuf; go.ldx0 = m->di; go.norm_w = ly.gnorm; go.eps = c.eps;
            if (with_attn) { go.W1 = ly.W_o; go.ldw1 = c.qh * c.hd; go.K1 = c.qh * c.hd; go.x1 = m->obuf; go.ldx1 = c.qh * c.hd; }
        } else if (ly.type == HS_LAYER_GDN) {
            go.W0 = ly.W_out; go.ldw0 = m->gw; go.K0 = m->gw; go.x0 = m->gbuf; go.ldx0 = m->gw;
        } else {
            go.W0 = ly.W_o; go.ldw0 = c.qh * c.hd; go.K0 = c.qh * c.hd; go.x0 = m->obuf; go.ldx0 = c.qh * c.hd;
        }
        go.early_trigger = 1; go.pf_ptr = ly.W_gu; go.pf_bytes = 2 * (int64_t)2 * c.ff * d;
        go.xb = m->xb; go.xb_rows = m->xb_rows;
        if (tc_pass) { go.pk_out = m->xb_h; go.pk_ld = d; go.pk_nw = ly.norm2; go.ss_out = m->ssbuf; }
        PROF(HS_PROF_GEMV, gemv_bytes(go), launch_gemv(go, st_w, s, &m->launches, &hparts), "out_proj");
        cur ^= 1;
        // (5) RMSNorm + gate/up + SwiGLU, (6) down + residual
        GemvArgs gu{};
        gu.W0 = ly.W_gu; gu.ldw0 = d; gu.K0 = d; gu.x0 = m->hbuf[cur]; gu.ldx0 = d; gu.xparts = hparts; gu.xpstride = hps;
        gu.norm_w = ly.norm2; gu.eps = c.eps;
        gu.O = 2 * c.ff; gu.out = m->abuf; gu.ldo = c.ff; gu.nrows = rows; gu.epi = EPI_SWIGLU;
        gu.early_trigger = 1; gu.pf_ptr = ly.W_down; gu.pf_bytes = 2 * (int64_t)d * c.ff;
        gu.xb = m->xb; gu.xb_rows = m->xb_rows;
        if (tc_pass) { gu.pk_in = m->xb_h; gu.ss_in = m->ssbuf; gu.ss_parts = ss_parts; gu.pk_out = m->xb_a; gu.pk_ld = c.ff; }
        PROF(HS_PROF_GEMV, gemv_bytes(gu), launch_gemv(gu, st_w, s, &m->launches, nullptr), "gate_up");
        GemvArgs gdn{};
        gdn.W0 = ly.W_down; gdn.ldw0 = c.ff; gdn.K0 = c.ff; gdn.x0 = m->abuf; gdn.ldx0 = c.ff; gdn.xparts = 1;
        gdn.O = d; gdn.out = m->hbuf[cur ^ 1]; gdn.ldo = d; gdn.opstride = hps; gdn.max_oparts = HS_H_PARTS;
        gdn.resid = m->hbuf[cur]; gdn.rparts = hparts; gdn.rpstride = hps; gdn.nrows = rows; gdn.epi = EPI_RESID;
        gdn.early_trigger = 1;
        {   // next projection in the chain: the following layer's in-projection, or the LM head
            int nl = l + 1;
            while (nl < c.L && draft && !draft_runs(m, nl)) ++nl;
            if (nl < c.L) {
                const bool na = m->layers[nl].type != HS_LAYER_GDN && (!draft || m->plan[nl] == HS_DRAFT_FULL);
                gdn.pf_ptr = m->layers[nl].W_in; gdn.pf_bytes = 2 * (int64_t)d * (na ? m->layers[nl].in_rows_full : m->layers[nl].in_rows_draft);
            }
            else { gdn.pf_ptr = m->lm_head; gdn.pf_bytes = 2 * (int64_t)c.V * d; }
            // the consumer of this layer's output: the next layer that runs (its first norm), else the final norm
            if (tc_pass) { gdn.pk_out = m->xb_h; gdn.pk_ld = d; gdn.pk_nw = nl < c.L ? m->layers[nl].norm1 : m->final_norm; gdn.ss_out = m->ssbuf; }
        }
        gdn.xb = m->xb; gdn.xb_rows = m->xb_rows;
        if (tc_pass) gdn.pk_in = m->xb_a;
        PROF(HS_PROF_GEMV, gemv_bytes(gdn), launch_gemv(gdn, st_w, s, &m->launches, &hparts), "down");
        cur ^= 1;
        h_packed = tc_pass;
    }
    if (!head) { m->last_rows = 0; return HS_OK; }       // the draft model only had to consume these positions
    // final norm + LM head, then greedy argmax
    GemvArgs lm{};
    lm.W0 = m->lm_head; lm.ldw0 = d; lm.K0 = d; lm.x0 = m->hbuf[cur]; lm.ldx0 = d; lm.xparts = hparts; lm.xpstride = hps;
    lm.norm_w = m->final_norm; lm.eps = c.eps;
    // a draft step at temperature > 0 keeps its logits (Eq. 6 needs P_S of every draft position at verification time)
    const bool sampled = draft && m->tau > 0.f;
    const int64_t dstride = (int64_t)std::max(c.max_k, 1) * c.V;
    lm.O = c.V; lm.nrows = rows; lm.epi = EPI_STORE;
    if (sampled) { lm.out = m->dlogits + (size_t)b0 * dstride + (size_t)step * c.V; lm.ldo = (int)dstride; }
    else { lm.out = m->logits; lm.ldo = c.V; }
    lm.early_trigger = 1;
    lm.xb = m->xb; lm.xb_rows = m->xb_rows;
    if (tc_pass && h_packed) { lm.pk_in = m->xb_h; lm.ss_in = m->ssbuf; lm.ss_parts = ss_parts; }
    PROF(HS_PROF_GEMV, gemv_bytes(lm), launch_gemv(lm, st_w, s, &m->launches, nullptr), "lm_head");
    if (sampled) PROF(HS_PROF_ARGMAX, 0, launch_sample(m->dlogits + (size_t)step * c.V, dstride, c.V, m->Tm, b0, nb, m->tau, m->u_draft, c.max_k, step,
                                                       m->ctrl.cand, step + 1, s), "draft draw");
    else if (draft) PROF(HS_PROF_ARGMAX, 0, launch_argmax(m->logits, c.V, 1, b0, nb, m->Tm, m->ctrl.cand, step + 1, nullptr, m->am_part, m->ctrl.am_counters, s), "argmax");
    else PROF(HS_PROF_ARGMAX, 0, launch_argmax(m->logits, c.V, T, b0, nb, m->Tm, m->ctrl.g, 0, m->ctrl.margin, m->am_part, m->ctrl.am_counters, s), "argmax");
    ++m->launches;
    m->last_rows = rows;
    return HS_OK;
}

int enqueue_draft(hs_model *m, int k, int b0, int nb) {
    // a draft that keeps attention reads, in a step's attention prologue, the scratch KV row the previous step wrote:
    // then every step opens in plain stream order
    for (int st = 0; st < k; ++st) { int rc = model_pass(m, true, 1, st, b0, nb, st == 0 || m->plan_attn); if (rc) return rc; }
    // literal draft state: the draft model must also have consumed the last candidate (d_k; the pending token when k = 0)
    // if the round accepts everything - one more step without the LM head
    if (m->literal) { int rc = model_pass(m, true, 1, k, b0, nb, k == 0, false, false); if (rc) return rc; }
    return HS_OK;
}

int enqueue_accept(hs_model *m, int k, int b0, int nb, const int32_t *fn, const int32_t *fx) {
    AcceptArgs a{};
    a.k = k; a.Tm = m->Tm; a.b0 = b0; a.nb = nb; a.n_rl = m->n_rl; a.B = m->B; a.convd = m->convd; a.V = m->c.V;
    a.ctrl = m->ctrl; a.forced_n = fn; a.forced_next = fx; a.cw = m->cw; a.hist = m->hist; a.replay = m->log_w != 0;
    if (m->literal) { a.dcw = m->dcwc; a.dhist = m->dhist; a.dslot = m->ctrl.dslot; a.dslot_mod = m->Tm + 1; }
    PROF(HS_PROF_ACCEPT, 0, launch_accept(a, m->stream), "accept");
    ++m->launches;
    if (m->log_w && m->n_rl > 0) {
        // rollback by replay: the accepted updates go into the committed state, every recurrent layer in one launch
        ReplayArgs r{};
        r.arch = m->c.arch; r.H = m->c.H; r.P = m->c.P; r.N = m->c.N; r.di = m->di; r.gh = m->c.gh; r.dk = m->c.gdk; r.dv = m->c.gdv;
        r.state = m->snap; r.log = m->ulog; r.log_w = m->log_w; r.n_acc = m->ctrl.n_acc; r.state_elems = m->state_elems;
        r.n_rl = m->n_rl; r.B = m->B; r.Tm = m->Tm; r.b0 = b0; r.nb = nb; r.status = m->ctrl.status;
        PROF(HS_PROF_ACCEPT, 0, launch_replay(r, m->stream), "replay");
        ++m->launches;
    }
    return HS_OK;
}

// Run `body` directly, or (HS_FLAG_GRAPHS) capture it once per key and replay the graph.
template <class F>
int run_maybe_graph(hs_model *m, uint64_t key, F body) {
    if (!(m->c.flags & HS_FLAG_GRAPHS) || m->prof) return body();
    auto it = m->graphs.find(key);
    if (it == m->graphs.end()) {
        int64_t before = m->launches;
        CK(cudaStreamBeginCapture(m->stream, cudaStreamCaptureModeThreadLocal), "begin capture");
        int rc = body();
        cudaGraph_t graph = nullptr;
        cudaError_t e = cudaStreamEndCapture(m->stream, &graph);
        if (rc != HS_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
        if (e != cudaSuccess) return cuda_fail(m, e, "end capture");
        cudaGraphExec_t exec = nullptr;
        e = cudaGraphInstantiate(&exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) return cuda_fail(m, e, "graph instantiate");
        m->graphs[key] = exec;
        m->graph_launches[key] = (int)(m->launches - before);
        m->launches = before;
        it = m->graphs.find(key);
    }
    CK(cudaGraphLaunch(it->second, m->stream), "graph launch");
    m->launches += m->graph_launches[key];
    return HS_OK;
}

int check_capacity(hs_model *m, int T, int b0, int nb) {
    for (int b = b0; b < b0 + nb; ++b)
        if (m->kv_upper[b] + T > m->c.kv_capacity) return fail(m, HS_ERR_CAPACITY, "kv_len + k + 1 exceeds kv_capacity");
    return HS_OK;
}

}  // namespace

// ================================================================================================
extern "C" {

int hs_query_sizes(const hs_config *cfg, hs_sizes *out) {
    if (!cfg || !out || !valid_config(*cfg)) return HS_ERR_INVALID_ARG;
    const hs_config &c = *cfg;
    Derived v = derive(c);
    out->weights = blob_offset(c, c.L, 0);
    out->snap = up((int64_t)4 * v.n_rl * v.B * (v.nslot * v.state_elems + (int64_t)v.Tm * v.log_w));
    out->dstate = up((int64_t)4 * v.n_rl * v.B * v.state_elems * (v.literal ? v.Tm + 1 : 1));
    out->conv = up((int64_t)4 * v.n_rl * v.B * v.convd * (3 + v.Tm + 6 + (v.literal ? 3 + v.Tm : 0)));
    out->kv = up((int64_t)2 * 2 * v.n_al * v.B * c.kvh * c.kv_capacity * c.hd);
    out->work = work_layout(c, v).total;
    return HS_OK;
}

int64_t hs_weight_offset(const hs_config *cfg, int layer, int tensor) {
    if (!cfg || !valid_config(*cfg) || layer < -1 || layer >= cfg->L) return -1;
    return blob_offset(*cfg, layer, tensor);
}

static int init_model(hs_model *m, const hs_config *cfg, const hs_buffers *bufs, void *stream);

int hs_init_model(const hs_config *cfg, const hs_buffers *bufs, const hs_sizes *have, void *stream, hs_model **out) {
    if (out) *out = nullptr;
    if (!cfg || !bufs || !have || !out || !valid_config(*cfg)) return HS_ERR_INVALID_ARG;
    const void *ptrs[6] = {bufs->weights, bufs->snap, bufs->dstate, bufs->conv, bufs->kv, bufs->work};
    for (int i = 0; i < 6; ++i) if (!ptrs[i] || ((uintptr_t)ptrs[i] & (ALIGN - 1))) return HS_ERR_INVALID_ARG;
    hs_sizes need;
    if (hs_query_sizes(cfg, &need) != HS_OK) return HS_ERR_INVALID_ARG;
    if (have->weights < need.weights || have->snap < need.snap || have->dstate < need.dstate || have->conv < need.conv ||
        have->kv < need.kv || have->work < need.work) return HS_ERR_SIZE;
    hs_model *m = new hs_model();
    const int rc = init_model(m, cfg, bufs, stream);
    if (rc != HS_OK) { delete m; return rc; }      // nothing is left behind by a failed call
    *out = m;
    return HS_OK;
}

static int init_model(hs_model *m, const hs_config *cfg, const hs_buffers *bufs, void *stream) {
    m->c = *cfg; m->bufs = *bufs; m->stream = (cudaStream_t)stream;
    const hs_config &c = m->c;
    Derived v = derive(c);
    m->B = v.B; m->Tm = v.Tm; m->batch = 0; m->di = d_inner(c); m->convd = v.convd; m->gw = v.gw;
    m->n_rl = v.n_rl; m->n_al = v.n_al; m->state_elems = v.state_elems; m->in_rows_max = v.in_rows_max;
    m->att_chunk = v.att_chunk; m->att_nch = v.att_nch; m->att_force_chunk = m->att_force_tiles = 0;
    m->nslot = v.nslot; m->log_w = v.log_w;
    m->phase = 0; m->last_k = -1; m->last_rows = 0; m->launches = 0; m->prof = false;
    m->kv_upper.assign(v.B, 0);
    const char *wb = (const char *)bufs->weights;
    auto f32 = [&](int l, int t) { int64_t o = blob_offset(c, l, t); return o < 0 ? nullptr : (const float *)(wb + o); };
    auto b16 = [&](int l, int t) { int64_t o = blob_offset(c, l, t); return o < 0 ? nullptr : (const __nv_bfloat16 *)(wb + o); };
    m->embed = b16(-1, HS_G_EMBED); m->lm_head = b16(-1, HS_G_LM_HEAD); m->final_norm = f32(-1, HS_G_FINAL_NORM);
    int rl = 0, al = 0;
    for (int l = 0; l < c.L; ++l) {
        HsLayer ly{};
        ly.type = layer_type(c, l);
        ly.rl = ly.type != HS_LAYER_ATT ? rl++ : -1;
        ly.al = ly.type != HS_LAYER_GDN ? al++ : -1;
        ly.norm1 = f32(l, HS_T_NORM1); ly.conv_w = f32(l, HS_T_CONV_W); ly.conv_b = f32(l, HS_T_CONV_B);
        ly.A_log = f32(l, HS_T_A_LOG); ly.D = f32(l, HS_T_D); ly.dt_bias = f32(l, HS_T_DT_BIAS);
        ly.gnorm = f32(l, HS_T_GNORM); ly.norm2 = f32(l, HS_T_NORM2);
        ly.W_in = b16(l, HS_T_W_IN); ly.W_out = b16(l, HS_T_W_OUT); ly.W_o = b16(l, HS_T_W_O);
        ly.W_gu = b16(l, HS_T_W_GU); ly.W_down = b16(l, HS_T_W_DOWN);
        ly.in_rows_full = in_rows(c, ly.type, false); ly.in_rows_draft = in_rows(c, ly.type, true);
        m->layers.push_back(ly);
    }
    m->plan.assign(c.L, HS_DRAFT_LINEAR); m->plan_attn = false; m->last_draft_k = 1;
    // carve the work buffer
    char *w = (char *)bufs->work;
    WorkLayout wl = work_layout(c, v);
    m->ctrl.kv_len = (int32_t *)(w + wl.kv_len); m->ctrl.slot = (int32_t *)(w + wl.slot);
    m->ctrl.cand = (int32_t *)(w + wl.cand); m->ctrl.g = (int32_t *)(w + wl.g); m->ctrl.margin = (float *)(w + wl.margin);
    m->ctrl.n_acc = (int32_t *)(w + wl.n_acc); m->ctrl.emitted = (int32_t *)(w + wl.emitted);
    m->ctrl.stage_n = (int32_t *)(w + wl.stage_n); m->ctrl.stage_next = (int32_t *)(w + wl.stage_next);
    m->ctrl.status = (int32_t *)(w + wl.status); m->ctrl.counters = (int32_t *)(w + wl.counters); m->ctrl.am_counters = (int32_t *)(w + wl.am_counters);
    m->ctrl.dslot = (int32_t *)(w + wl.dslot);
    m->rope = (float2 *)(w + wl.rope);
    m->hbuf[0] = (float *)(w + wl.h); m->hbuf[1] = m->hbuf[0] + (size_t)HS_H_PARTS * v.R * c.d; m->zx = (float *)(w + wl.zx); m->gbuf = (float *)(w + wl.gbuf);
    m->obuf = (float *)(w + wl.obuf); m->abuf = (float *)(w + wl.abuf); m->logits = (float *)(w + wl.logits); m->dlogits = (float *)(w + wl.dlogits);
    m->tau = 0.f; m->u_draft = m->u_accept = m->u_final = nullptr;
    m->att_acc = (float *)(w + wl.att_acc); m->att_ml = (float *)(w + wl.att_ml); m->am_part = w + wl.am_part; m->xb = (__nv_bfloat16 *)(w + wl.xb); m->xb_rows = gemm_tc_rows(v.R);
    m->xb_h = (__nv_bfloat16 *)(w + wl.xb_h); m->xb_a = (__nv_bfloat16 *)(w + wl.xb_a); m->ssbuf = (float *)(w + wl.ssbuf);
    // the tcgen05 kernel's fixed cost (operand packing, tensor-memory set-up, epilogue out of tensor memory) pays from
    // 7 activation rows on, from 4 where the weight matrices are large (measured: model widths 1024 and 2560)
    m->tc_min_rows_auto = (int64_t)4 * c.ff * c.d >= ((int64_t)64 << 20) ? 4 : 7;
    g_hs_tc_min_rows = m->tc_min_rows_auto;
    // conv buffer: committed windows | verify history | draft ping-pong
    float *cv = (float *)bufs->conv;
    const size_t win = (size_t)v.n_rl * v.B * 3 * v.convd;
    m->cw = cv; m->hist = cv + win; m->dcw = m->hist + (size_t)v.n_rl * v.B * v.Tm * v.convd;
    m->literal = v.literal != 0;
    m->dcwc = m->dcw + 2 * win; m->dhist = m->dcwc + win;        // used with the literal draft state only
    m->Kc = (__nv_bfloat16 *)bufs->kv;
    m->Vc = m->Kc + (size_t)v.n_al * v.B * c.kvh * c.kv_capacity * c.hd;
    m->snap = (float *)bufs->snap; m->dstate = (float *)bufs->dstate;
    m->ulog = m->log_w ? m->snap + (size_t)v.n_rl * v.B * v.nslot * v.state_elems : nullptr;
    CK(configure_gemv(), "configure gemv");
    CK(configure_attn(), "configure attention");
    if (configure_gemm_tc() != cudaSuccess) { g_hs_gemm_tc = false; cudaGetLastError(); }   // falls back to several 16-row launches
    if (g_hs_tensor_maps && c.hd % 64 == 0) {     // tensor maps of every attention layer's cache (streaming attention form)
        const size_t per_layer = (size_t)v.B * c.kvh * c.kv_capacity * c.hd;
        m->kmaps.resize(v.n_al); m->vmaps.resize(v.n_al);
        for (int al = 0; al < v.n_al; ++al)
            if (hs_make_kv_tensor_map(&m->kmaps[al], m->Kc + al * per_layer, (uint64_t)v.B * c.kvh * c.kv_capacity, c.hd) != cudaSuccess ||
                hs_make_kv_tensor_map(&m->vmaps[al], m->Vc + al * per_layer, (uint64_t)v.B * c.kvh * c.kv_capacity, c.hd) != cudaSuccess) {
                m->kmaps.clear(); m->vmaps.clear(); cudaGetLastError();
                break;
            }
    }
    // RoPE table (rotate-half pairing: pair (e, e + hd/2) turns by pos * theta^(-2e/hd)), computed in double
    std::vector<float2> tab((size_t)c.kv_capacity * (c.hd / 2));
    for (int e = 0; e < c.hd / 2; ++e) {
        const double f = std::pow((double)c.rope_theta, -2.0 * e / c.hd);
        for (int p = 0; p < c.kv_capacity; ++p) {
            const double ang = (double)p * f;
            tab[(size_t)p * (c.hd / 2) + e] = make_float2((float)std::cos(ang), (float)std::sin(ang));
        }
    }
    CK(cudaMemcpyAsync(m->rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, m->stream), "rope upload");
    CK(cudaMemsetAsync(w, 0, wl.rope, m->stream), "ctrl clear");
    CK(cudaStreamSynchronize(m->stream), "init sync");
    return HS_OK;
}

int hs_reset(hs_model *m) {
    if (!m) return HS_ERR_INVALID_ARG;
    hs_sizes sz; hs_query_sizes(&m->c, &sz);
    CK(cudaMemsetAsync(m->snap, 0, sz.snap, m->stream), "reset snap");
    CK(cudaMemsetAsync(m->dstate, 0, sz.dstate, m->stream), "reset dstate");
    CK(cudaMemsetAsync(m->bufs.conv, 0, sz.conv, m->stream), "reset conv");
    CK(cudaMemsetAsync(m->bufs.work, 0, (char *)m->rope - (char *)m->bufs.work, m->stream), "reset ctrl");
    std::fill(m->kv_upper.begin(), m->kv_upper.end(), 0);
    m->phase = 0; m->batch = 0;
    return HS_OK;
}

int hs_set_batch(hs_model *m, int batch) {
    if (!m || batch < 1 || batch > m->B) return HS_ERR_INVALID_ARG;
    m->batch = batch; m->phase = 0;
    return HS_OK;
}

int hs_prefill(hs_model *m, const int32_t *tokens_host, const int32_t *lens_host, int batch) {
    if (!m || !tokens_host || !lens_host || batch < 1 || batch > m->B) return HS_ERR_INVALID_ARG;
    int64_t off = 0;
    for (int b = 0; b < batch; ++b) {
        if (lens_host[b] < 1) return fail(m, HS_ERR_INVALID_ARG, "empty prompt");
        if (m->kv_upper[b] + lens_host[b] > m->c.kv_capacity) return fail(m, HS_ERR_CAPACITY, "prompt exceeds kv_capacity");
        for (int p = 0; p < lens_host[b]; ++p)
            if (tokens_host[off + p] < 0 || tokens_host[off + p] >= m->c.V) return fail(m, HS_ERR_INVALID_ARG, "prompt token id outside [0, V)");
        off += lens_host[b];
    }
    // Chunk c covers prompt positions [c * Tm, (c + 1) * Tm) of every sequence that reaches that far; neighbouring
    // sequences with the same number of tokens in the chunk go out as one verify pass with every candidate accepted.
    // Nothing waits on the host between chunks (the token slices and accept lengths are staged by the copies).
    std::vector<int64_t> start(batch);
    int maxlen = 0;
    off = 0;
    for (int b = 0; b < batch; ++b) { start[b] = off; off += lens_host[b]; maxlen = std::max(maxlen, lens_host[b]); }
    std::vector<std::vector<int32_t>> acc_lens;           // alive until the final synchronisation
    for (int p = 0; p < maxlen; p += m->Tm) {
        acc_lens.emplace_back(batch, 0);
        std::vector<int32_t> &n = acc_lens.back();
        std::vector<int> Tb(batch);
        for (int b = 0; b < batch; ++b) {
            Tb[b] = std::max(0, std::min(m->Tm, lens_host[b] - p));
            n[b] = Tb[b] - 1;
            if (Tb[b] > 0)
                CK(cudaMemcpyAsync(m->ctrl.cand + b * m->Tm, tokens_host + start[b] + p, sizeof(int32_t) * Tb[b],
                                   cudaMemcpyHostToDevice, m->stream), "prefill tokens");
        }
        CK(cudaMemcpyAsync(m->ctrl.stage_n, n.data(), sizeof(int32_t) * batch, cudaMemcpyHostToDevice, m->stream), "prefill accept lengths");
        for (int b0 = 0; b0 < batch;) {
            int nb = 1;
            while (b0 + nb < batch && Tb[b0 + nb] == Tb[b0]) ++nb;
            if (Tb[b0] > 0) {
                int rc = model_pass(m, false, Tb[b0], 0, b0, nb, true);
                if (rc) return rc;
                if (m->literal) { rc = model_pass(m, true, Tb[b0], 0, b0, nb, true, true, false); if (rc) return rc; }
                rc = enqueue_accept(m, Tb[b0] - 1, b0, nb, m->ctrl.stage_n, nullptr);
                if (rc) return rc;
                for (int b = b0; b < b0 + nb; ++b) m->kv_upper[b] += Tb[b0];
            }
            b0 += nb;
        }
    }
    CK(cudaStreamSynchronize(m->stream), "prefill sync");   // host temporaries and the caller's tokens were read by now
    m->batch = batch; m->phase = 0;
    return hs_device_status(m);
}

int hs_draft(hs_model *m, int k) {
    if (!m || k < 0 || k > m->c.max_k) return HS_ERR_INVALID_ARG;
    if (m->batch < 1) return fail(m, HS_ERR_ORDER, "no active sequences: prefill or set_context first");
    if (m->phase == 2) return fail(m, HS_ERR_ORDER, "draft after verify: the snapshots hold the verified positions until accept_rollback");
    if (k > 0 || m->literal) {
        const int nb = m->batch;
        m->last_draft_k = k;
        uint64_t geo = 0;
        if (m->plan_attn) {         // scratch KV rows kv_len .. kv_len + k - 1
            int rc = check_capacity(m, k, 0, nb);
            if (rc) return rc;
            geo = (uint64_t)attn_geom(m, 1, k, 0, nb).code();
        }
        int rc = run_maybe_graph(m, (1ull << 60) | (geo << 32) | ((uint64_t)k << 20) | nb, [&] { return enqueue_draft(m, k, 0, nb); });
        if (rc) return rc;
    }
    m->phase = 1; m->last_k = k;
    m->sampled_draft = m->tau > 0.f;
    return HS_OK;
}

int hs_verify(hs_model *m, int k, const int32_t *cand_dev) {
    if (!m || k < 0 || k > m->c.max_k) return HS_ERR_INVALID_ARG;
    if (m->batch < 1) return fail(m, HS_ERR_ORDER, "no active sequences: prefill or set_context first");
    if (m->phase == 2) return fail(m, HS_ERR_ORDER, "verify after verify: the snapshots hold the verified positions until accept_rollback");
    if (!cand_dev && k > 0 && !(m->phase == 1 && m->last_k == k)) return fail(m, HS_ERR_ORDER, "verify(k) needs a preceding draft(k) or explicit candidates");
    const int nb = m->batch, T = k + 1;
    int rc = check_capacity(m, T, 0, nb);
    if (rc) return rc;
    if (cand_dev) m->sampled_draft = false;      // the kept draft distributions belong to other candidates
    if (cand_dev)
        CK(cudaMemcpy2DAsync(m->ctrl.cand, sizeof(int32_t) * m->Tm, cand_dev, sizeof(int32_t) * T, sizeof(int32_t) * T, nb,
                             cudaMemcpyDeviceToDevice, m->stream), "candidates");
    if (m->literal && (cand_dev || m->phase != 1)) {
        // the draft model's own state must follow the candidates that are verified, not the ones it drafted (or none)
        rc = model_pass(m, true, T, 0, 0, nb, true, true, false);
        if (rc) return rc;
    }
    rc = run_maybe_graph(m, (2ull << 60) | ((uint64_t)attn_geom(m, T, T, 0, nb).code() << 32) | ((uint64_t)k << 20) | nb, [&] { return model_pass(m, false, T, 0, 0, nb, true); });
    if (rc) return rc;
    m->phase = 2; m->last_k = k;
    return HS_OK;
}

int hs_accept_rollback(hs_model *m, const int32_t *forced_n_dev, const int32_t *forced_next_dev,
                       int32_t *n_acc_host, int32_t *emitted_host) {
    if (!m) return HS_ERR_INVALID_ARG;
    if (m->phase != 2) return fail(m, HS_ERR_ORDER, "accept_rollback needs a preceding verify");
    const int k = m->last_k, nb = m->batch, T = k + 1;
    if (m->tau > 0.f && !forced_n_dev) {
        // Eq. 6: the accept length and the correction / bonus token are drawn on the device, then applied like forced ones
        if (!m->sampled_draft && k > 0) return fail(m, HS_ERR_ORDER, "sampling needs the draft distributions of this round: hs_draft at the same temperature, or forced accept lengths");
        PROF(HS_PROF_ACCEPT, 0, launch_spec_accept(m->dlogits, (int64_t)std::max(m->c.max_k, 1) * m->c.V, m->logits, m->ctrl.cand, m->u_accept, m->u_final,
                                                   m->c.max_k, m->ctrl.stage_n, m->ctrl.stage_next, m->c.V, m->Tm, k, 0, nb, m->tau, m->stream), "sampled accept");
        ++m->launches;
        forced_n_dev = m->ctrl.stage_n;
        if (!forced_next_dev) forced_next_dev = m->ctrl.stage_next;
    }
    int rc = enqueue_accept(m, k, 0, nb, forced_n_dev, forced_next_dev);
    if (rc) return rc;
    m->phase = 0;
    for (int b = 0; b < nb; ++b) m->kv_upper[b] += T;
    if (n_acc_host || emitted_host) {
        std::vector<int32_t> n(nb);
        CK(cudaMemcpyAsync(n.data(), m->ctrl.n_acc, 4 * nb, cudaMemcpyDeviceToHost, m->stream), "n_acc readback");
        if (emitted_host)
            CK(cudaMemcpy2DAsync(emitted_host, 4 * T, m->ctrl.emitted, 4 * m->Tm, 4 * T, nb, cudaMemcpyDeviceToHost, m->stream), "emitted readback");
        CK(cudaStreamSynchronize(m->stream), "accept sync");
        for (int b = 0; b < nb; ++b) { m->kv_upper[b] += n[b] + 1 - T; if (n_acc_host) n_acc_host[b] = n[b]; }
    }
    return HS_OK;
}

int hs_round_host(hs_model *m, int k, const int32_t *forced_n_host, const int32_t *forced_next_host,
                  int32_t *n_acc_host, int32_t *emitted_host) {
    if (!m) return HS_ERR_INVALID_ARG;
    const int nb = m->batch;
    if (nb < 1) return fail(m, HS_ERR_ORDER, "no active sequences");
    if (k < 0 || k > m->c.max_k) return HS_ERR_INVALID_ARG;
    if (m->phase == 2) return fail(m, HS_ERR_ORDER, "round after verify: call accept_rollback first");
    if (forced_n_host)
        for (int b = 0; b < nb; ++b)
            if (forced_n_host[b] < 0 || forced_n_host[b] > k) return fail(m, HS_ERR_INVALID_ARG, "forced accept length outside [0, k]");
    if (forced_next_host)
        for (int b = 0; b < nb; ++b)
            if (forced_next_host[b] >= m->c.V) return fail(m, HS_ERR_INVALID_ARG, "forced next token id >= V");
    if (forced_n_host) CK(cudaMemcpyAsync(m->ctrl.stage_n, forced_n_host, 4 * nb, cudaMemcpyHostToDevice, m->stream), "forced_n upload");
    if (forced_next_host) CK(cudaMemcpyAsync(m->ctrl.stage_next, forced_next_host, 4 * nb, cudaMemcpyHostToDevice, m->stream), "forced_next upload");
    int rc = hs_draft(m, k);
    if (rc) return rc;
    rc = hs_verify(m, k, nullptr);
    if (rc) return rc;
    rc = hs_accept_rollback(m, forced_n_host ? m->ctrl.stage_n : nullptr, forced_next_host ? m->ctrl.stage_next : nullptr,
                            n_acc_host, emitted_host);
    if (rc) return rc;
    if (!n_acc_host && !emitted_host) CK(cudaStreamSynchronize(m->stream), "round sync");
    return HS_OK;
}

// ---- hooks ----------------------------------------------------------------------------------
static int state_xfer(hs_model *m, int layer, int seq, int kind, void *host, int64_t bytes, bool to_host) {
    if (!m || !host || layer < 0 || layer >= m->c.L || seq < 0 || seq >= m->B) return HS_ERR_INVALID_ARG;
    const hs_config &c = m->c;
    const HsLayer &ly = m->layers[layer];
    const cudaMemcpyKind dir = to_host ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice;
    CK(cudaStreamSynchronize(m->stream), "hook sync");
    if (kind == HS_STATE_SSM || kind == HS_STATE_GDN || kind == HS_STATE_DRAFT) {
        if (ly.rl < 0) return fail(m, HS_ERR_INVALID_ARG, "layer has no recurrent state");
        if (kind == HS_STATE_SSM && ly.type != HS_LAYER_PAR) return HS_ERR_INVALID_ARG;
        if (kind == HS_STATE_GDN && ly.type != HS_LAYER_GDN) return HS_ERR_INVALID_ARG;
        if (bytes != 4 * m->state_elems) return fail(m, HS_ERR_SIZE, "state size mismatch");
        float *dev;
        if (kind == HS_STATE_DRAFT) {
            if (!to_host) return HS_ERR_INVALID_ARG;
            if (m->literal) {
                int32_t ds = 0;
                CK(cudaMemcpy(&ds, m->ctrl.dslot + seq, 4, cudaMemcpyDeviceToHost), "draft slot read");
                dev = m->dstate + (((size_t)ly.rl * m->B + seq) * (m->Tm + 1) + ds) * m->state_elems;
            } else dev = m->dstate + ((size_t)ly.rl * m->B + seq) * m->state_elems;
        } else {
            int32_t slot = 0;
            if (to_host) CK(cudaMemcpy(&slot, m->ctrl.slot + seq, 4, cudaMemcpyDeviceToHost), "slot read");
            else CK(cudaMemcpy(m->ctrl.slot + seq, &slot, 4, cudaMemcpyHostToDevice), "slot write");
            dev = m->snap + (((size_t)ly.rl * m->B + seq) * m->nslot + (m->log_w ? 0 : slot)) * m->state_elems;
        }
        CK(to_host ? cudaMemcpy(host, dev, bytes, dir) : cudaMemcpy(dev, host, bytes, dir), "state copy");
        return HS_OK;
    }
    if (kind == HS_STATE_CONV || kind == HS_STATE_DRAFT_CONV) {
        if (ly.rl < 0) return fail(m, HS_ERR_INVALID_ARG, "layer has no conv window");
        if (kind == HS_STATE_DRAFT_CONV && (!m->literal || !to_host)) return HS_ERR_INVALID_ARG;
        if (bytes != (int64_t)4 * 3 * m->convd) return fail(m, HS_ERR_SIZE, "conv window size mismatch");
        float *dev = (kind == HS_STATE_CONV ? m->cw : m->dcwc) + ((size_t)ly.rl * m->B + seq) * 3 * m->convd;
        CK(to_host ? cudaMemcpy(host, dev, bytes, dir) : cudaMemcpy(dev, host, bytes, dir), "conv copy");
        return HS_OK;
    }
    if (kind == HS_STATE_K || kind == HS_STATE_V) {
        if (ly.al < 0) return fail(m, HS_ERR_INVALID_ARG, "layer has no KV cache");
        const int64_t rowb = (int64_t)c.kvh * c.hd * 2;
        if (bytes <= 0 || bytes % rowb) return fail(m, HS_ERR_SIZE, "KV bytes must be whole rows");
        const int64_t rows = bytes / rowb;
        if (rows > c.kv_capacity) return fail(m, HS_ERR_SIZE, "more rows than kv_capacity");
        __nv_bfloat16 *base = (kind == HS_STATE_K ? m->Kc : m->Vc) + ((size_t)ly.al * m->B + seq) * c.kvh * c.kv_capacity * c.hd;
        // device [kvh][cap][hd]  <->  host [rows][kvh][hd]
        for (int h = 0; h < c.kvh; ++h) {
            __nv_bfloat16 *dev = base + (size_t)h * c.kv_capacity * c.hd;
            char *hp = (char *)host + (size_t)h * c.hd * 2;
            if (to_host) CK(cudaMemcpy2D(hp, rowb, dev, c.hd * 2, c.hd * 2, rows, dir), "kv export");
            else CK(cudaMemcpy2D(dev, c.hd * 2, hp, rowb, c.hd * 2, rows, dir), "kv import");
        }
        return HS_OK;
    }
    return HS_ERR_INVALID_ARG;
}

int hs_export_state(hs_model *m, int layer, int seq, int kind, void *host, int64_t bytes) {
    return state_xfer(m, layer, seq, kind, host, bytes, true);
}
int hs_import_state(hs_model *m, int layer, int seq, int kind, const void *host, int64_t bytes) {
    return state_xfer(m, layer, seq, kind, const_cast<void *>(host), bytes, false);
}

int hs_set_context(hs_model *m, int seq, int kv_len, int pending) {
    if (!m || seq < 0 || seq >= m->B || kv_len < 0 || kv_len > m->c.kv_capacity || pending < 0 || pending >= m->c.V)
        return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "hook sync");
    int32_t v = kv_len, p = pending;
    CK(cudaMemcpy(m->ctrl.kv_len + seq, &v, 4, cudaMemcpyHostToDevice), "set kv_len");
    CK(cudaMemcpy(m->ctrl.cand + seq * m->Tm, &p, 4, cudaMemcpyHostToDevice), "set pending");
    m->kv_upper[seq] = kv_len;
    if (m->batch < seq + 1) m->batch = seq + 1;
    m->phase = 0;
    return HS_OK;
}

int hs_poke_control(hs_model *m, int seq, int word, int32_t value) {
    if (!m || seq < 0 || seq >= m->B || (word != HS_CTRL_KV_LEN && word != HS_CTRL_SLOT)) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "hook sync");
    int32_t *dst = (word == HS_CTRL_KV_LEN ? m->ctrl.kv_len : m->ctrl.slot) + seq;
    CK(cudaMemcpy(dst, &value, 4, cudaMemcpyHostToDevice), "poke control word");
    return HS_OK;
}

int hs_get_context(hs_model *m, int seq, int32_t *kv_len, int32_t *pending) {
    if (!m || seq < 0 || seq >= m->B) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "hook sync");
    int32_t v = 0, p = 0;
    CK(cudaMemcpy(&v, m->ctrl.kv_len + seq, 4, cudaMemcpyDeviceToHost), "get kv_len");
    CK(cudaMemcpy(&p, m->ctrl.cand + seq * m->Tm, 4, cudaMemcpyDeviceToHost), "get pending");
    if (m->phase == 0) m->kv_upper[seq] = v;
    if (kv_len) *kv_len = v;
    if (pending) *pending = p;
    return HS_OK;
}

int hs_get_logits(hs_model *m, float *host, int rows) {
    if (!m || !host || rows < 1 || rows > m->last_rows) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "hook sync");
    CK(cudaMemcpy(host, m->logits, (size_t)4 * rows * m->c.V, cudaMemcpyDeviceToHost), "logits");
    return HS_OK;
}

int hs_get_round(hs_model *m, int32_t *cand_host, int32_t *g_host, float *margin_host) {
    if (!m || m->last_k < 0 || m->batch < 1) return HS_ERR_INVALID_ARG;
    const int T = m->last_k + 1, nb = m->batch;
    CK(cudaStreamSynchronize(m->stream), "hook sync");
    if (cand_host) CK(cudaMemcpy2D(cand_host, 4 * T, m->ctrl.cand, 4 * m->Tm, 4 * T, nb, cudaMemcpyDeviceToHost), "cand");
    if (g_host) CK(cudaMemcpy2D(g_host, 4 * T, m->ctrl.g, 4 * m->Tm, 4 * T, nb, cudaMemcpyDeviceToHost), "g");
    if (margin_host) CK(cudaMemcpy2D(margin_host, 4 * T, m->ctrl.margin, 4 * m->Tm, 4 * T, nb, cudaMemcpyDeviceToHost), "margin");
    return HS_OK;
}

int64_t hs_launch_count(const hs_model *m) { return m ? m->launches : -1; }

int hs_set_attn_geometry(hs_model *m, int chunk, int tiles) {
    if (!m) return HS_ERR_INVALID_ARG;
    if (chunk == 0) { m->att_force_chunk = m->att_force_tiles = 0; return HS_OK; }
    if (tiles < 0) {        // the streaming form: 128-key tiles, -tiles of them per CTA
        if (chunk != 128 || tiles < -32 || (m->c.qh / m->c.kvh) * (m->c.max_k + 1) > 32)
            return fail(m, HS_ERR_INVALID_ARG, "streaming attention: chunk 128, 1..32 tiles, at most 32 query rows per KV head");
        if (m->kmaps.empty()) return fail(m, HS_ERR_INVALID_ARG, "streaming attention needs the driver's tensor-map encoder and a head dimension that is a multiple of 64");
    } else if (chunk < 16 || chunk > 128 || (chunk & 15) || tiles < 1 || tiles > 32 || chunk * tiles < m->att_chunk)
        return fail(m, HS_ERR_INVALID_ARG, "attention geometry: chunk a multiple of 16 up to 128, tiles 1..32, chunk * tiles >= workspace chunk");
    m->att_force_chunk = chunk; m->att_force_tiles = tiles;
    return HS_OK;
}

int hs_set_draft_plan(hs_model *m, const int32_t *plan_host) {
    if (!m) return HS_ERR_INVALID_ARG;
    if (m->phase == 1) return fail(m, HS_ERR_ORDER, "the draft plan cannot change between a draft and its verification");
    std::vector<int> plan(m->c.L, HS_DRAFT_LINEAR);
    bool attn = false;
    if (plan_host)
        for (int l = 0; l < m->c.L; ++l) {
            if (plan_host[l] < HS_DRAFT_SKIP || plan_host[l] > HS_DRAFT_FULL) return fail(m, HS_ERR_INVALID_ARG, "draft plan entries are HS_DRAFT_SKIP, _LINEAR or _FULL");
            plan[l] = plan_host[l];
            if (plan[l] == HS_DRAFT_FULL && m->layers[l].type != HS_LAYER_GDN) attn = true;
        }
    if (attn && m->literal) return fail(m, HS_ERR_INVALID_ARG, "the literal draft state goes with draft plans that keep no attention");
    CK(cudaStreamSynchronize(m->stream), "plan sync");
    m->plan = plan; m->plan_attn = attn;
    for (auto &kv : m->graphs) cudaGraphExecDestroy(kv.second);     // the draft graphs were captured for the old plan
    m->graphs.clear(); m->graph_launches.clear();
    return HS_OK;
}

int hs_set_sampling(hs_model *m, float temperature, const float *u_draft_dev, const float *u_accept_dev, const float *u_final_dev) {
    if (!m) return HS_ERR_INVALID_ARG;
    if (m->phase != 0) return fail(m, HS_ERR_ORDER, "the sampling mode changes between rounds only");
    const bool on = temperature > 0.f;
    if (on && (!u_draft_dev || !u_accept_dev || !u_final_dev)) return fail(m, HS_ERR_INVALID_ARG, "sampling needs the three uniform arrays");
    if (!(temperature >= 0.f)) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "sampling sync");
    m->tau = on ? temperature : 0.f;
    m->u_draft = on ? u_draft_dev : nullptr; m->u_accept = on ? u_accept_dev : nullptr; m->u_final = on ? u_final_dev : nullptr;
    m->sampled_draft = false;
    for (auto &kv : m->graphs) cudaGraphExecDestroy(kv.second);     // the draft graphs depend on the mode and the pointers
    m->graphs.clear(); m->graph_launches.clear();
    return HS_OK;
}

int hs_set_option(hs_model *m, int option, int value) {
    if (!m) return HS_ERR_INVALID_ARG;
    if (option == HS_OPT_TC_MIN_ROWS) {
        if (value != 0 && (value < 2 || value > 17)) return fail(m, HS_ERR_INVALID_ARG, "tcgen05 row threshold out of range");
        CK(cudaStreamSynchronize(m->stream), "option sync");
        g_hs_tc_min_rows = value ? value : m->tc_min_rows_auto;
        for (auto &kv : m->graphs) cudaGraphExecDestroy(kv.second);
        m->graphs.clear(); m->graph_launches.clear();
        return HS_OK;
    }
    bool *flag = option == HS_OPT_CLUSTER_REDUCE ? &g_hs_cluster_reduce : option == HS_OPT_GEMM_MMA ? &g_hs_gemm_mma
               : option == HS_OPT_GEMM_TC ? &g_hs_gemm_tc : option == HS_OPT_PDL ? &g_hs_pdl
               : option == HS_OPT_ATTN_SMALL ? &g_hs_attn_small : option == HS_OPT_ATTN_STREAM ? &g_hs_attn_stream : nullptr;
    if (!flag) return fail(m, HS_ERR_INVALID_ARG, "unknown option");
    CK(cudaStreamSynchronize(m->stream), "option sync");
    *flag = value != 0;
    for (auto &kv : m->graphs) cudaGraphExecDestroy(kv.second);     // captured with the old choice
    m->graphs.clear(); m->graph_launches.clear();
    return HS_OK;
}

int hs_profile(hs_model *m, int enable) {
    if (!m) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "profile sync");
    for (auto &e : m->prof_events) { cudaEventDestroy(e.start); if (e.stop) cudaEventDestroy(e.stop); }
    m->prof_events.clear();
    m->prof = enable != 0;
    return HS_OK;
}

int hs_profile_read(hs_model *m, double *ms, int64_t *launches, double *bytes) {
    if (!m || !ms || !launches || !bytes) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "profile sync");
    for (int i = 0; i < HS_PROF_COUNT; ++i) { ms[i] = 0; launches[i] = 0; bytes[i] = 0; }
    for (auto &e : m->prof_events) {
        if (!e.stop) continue;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, e.start, e.stop) != cudaSuccess) continue;
        ms[e.cat] += t; launches[e.cat] += 1; bytes[e.cat] += e.bytes;
    }
    return HS_OK;
}

int hs_device_status(hs_model *m) {
    if (!m) return HS_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(m->stream), "status sync");
    int32_t st = 0;
    CK(cudaMemcpy(&st, m->ctrl.status, 4, cudaMemcpyDeviceToHost), "status read");
    if (st != 0) { m->err = "a kernel recorded an error in the device status word"; return st; }
    return HS_OK;
}

int hs_selftest_wait_timeout(hs_model *m, int polls) {
    if (!m || polls < 1 || polls > (1 << 20)) return HS_ERR_INVALID_ARG;
    CK(launch_wait_probe(m->ctrl.status, polls, m->stream), "wait probe");
    ++m->launches;
    return HS_OK;
}

int hs_clear_status(hs_model *m) {
    if (!m) return HS_ERR_INVALID_ARG;
    CK(cudaMemsetAsync(m->ctrl.status, 0, 4, m->stream), "status clear");
    return HS_OK;
}

const char *hs_last_error(const hs_model *m) { return m ? m->err.c_str() : "null handle"; }

int hs_destroy(hs_model *m) {
    if (!m) return HS_ERR_INVALID_ARG;
    for (auto &kv : m->graphs) cudaGraphExecDestroy(kv.second);
    for (auto &e : m->prof_events) { cudaEventDestroy(e.start); if (e.stop) cudaEventDestroy(e.stop); }
    delete m;
    return HS_OK;
}

}  // extern "C"

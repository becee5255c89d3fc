// Small kernels of the round: token embedding gather, greedy argmax with top-2 margin, and the
// accept / rollback step (paper Sec. 3.3, greedy rule).
#include "hs_internal.h"
#include "hs_device.cuh"
#include <mutex>

bool g_hs_pdl = true;

namespace {
using namespace hsd;

// h[row(b,i)][:] = E[cand[b][col0 + i]].  A token id outside [0, V) (a caller's candidate buffer, a forced
// next token) is never used as an address: the row of token 0 is gathered instead and the status word is set.
__global__ void embed_kernel(const __nv_bfloat16 *E, int d, int V, const int32_t *cand, int Tm, int col0, int T,
                             int b0, float *h, int32_t *status) {
    const int i = blockIdx.x, lb = blockIdx.y, b = b0 + lb;
    pdl_trigger();
    pdl_wait();
    int tok = __ldcg(cand + b * Tm + col0 + i);
    if (tok < 0 || tok >= V) {
        if (threadIdx.x == 0) atomicCAS(status, 0, (int)HS_ERR_DEVICE);
        tok = 0;
    }
    const uint4 *src = reinterpret_cast<const uint4 *>(E + (size_t)tok * d);
    float *dst = h + (size_t)(lb * T + i) * d;
    for (int c = threadIdx.x; c < d / 8; c += blockDim.x) {
        uint4 w = src[c];
        float4 lo = make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u),
                                __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
        float4 hi = make_float4(__uint_as_float(w.z << 16), __uint_as_float(w.z & 0xffff0000u),
                                __uint_as_float(w.w << 16), __uint_as_float(w.w & 0xffff0000u));
        reinterpret_cast<float4 *>(dst)[2 * c] = lo;
        reinterpret_cast<float4 *>(dst)[2 * c + 1] = hi;
    }
}

struct Top2 { float v1; int i1; float v2; };

__device__ __forceinline__ Top2 top2_merge(const Top2 &a, const Top2 &b) {
    // lowest index wins a tie for first place; an equal runner-up makes the margin zero
    Top2 r;
    if (a.v1 > b.v1 || (a.v1 == b.v1 && a.i1 < b.i1)) { r.v1 = a.v1; r.i1 = a.i1; r.v2 = fmaxf(a.v2, b.v1); }
    else { r.v1 = b.v1; r.i1 = b.i1; r.v2 = fmaxf(b.v2, a.v1); }
    return r;
}

// Greedy argmax with top-2 margin over V logits per row, split over HS_ARGMAX_CHUNKS CTAs per row.
// grid = (chunks, T, nb).  A CTA scans its slice (lowest id wins a tie), writes a partial
// (top value, its id, runner-up) to scratch and takes a ticket; the CTA that arrives last merges the
// row's partials - the merge is order-independent, so the result is reproducible - writes the token
// and the margin and puts the ticket counter back to zero for the next launch.
struct ArgmaxArgs {
    const float *logits; int V, T, b0, Tm;
    int32_t *tok_out; int tok_col0; float *margin_out;
    float4 *part;            // scratch [rows][HS_ARGMAX_CHUNKS]
    int32_t *counters;       // scratch [rows], zero between launches
};

__device__ __forceinline__ Top2 top2_warp(Top2 t) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        Top2 u;
        u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, u);
    }
    return t;
}

__global__ void __launch_bounds__(256) argmax_kernel(const ArgmaxArgs a) {
    const int chunk = blockIdx.x, i = blockIdx.y, lb = blockIdx.z, b = a.b0 + lb;
    const int nchunk = gridDim.x;
    const float *row = a.logits + (size_t)(lb * a.T + i) * a.V;
    const int srow = b * a.Tm + i;                                // scratch slot of this logits row
    const int per = ((a.V + nchunk - 1) / nchunk + 3) & ~3;
    const int lo = chunk * per, hi = min(a.V, lo + per);
    pdl_trigger();
    pdl_wait();
    Top2 t = {-INFINITY, 0x7fffffff, -INFINITY};
    auto feed = [&](float v, int j) {
        if (v > t.v1) { t.v2 = t.v1; t.v1 = v; t.i1 = j; }
        else if (v > t.v2) t.v2 = v;
    };
    if ((a.V & 3) == 0) {
        for (int j = lo + threadIdx.x * 4; j < hi; j += blockDim.x * 4) {
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(row + j));
            feed(v.x, j); feed(v.y, j + 1); feed(v.z, j + 2); feed(v.w, j + 3);
        }
    } else {
        for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) feed(__ldcg(row + j), j);
    }
    t = top2_warp(t);
    __shared__ Top2 s[8];
    __shared__ int ticket_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) s[warp] = t;
    __syncthreads();
    if (warp != 0) return;
    t = lane < (int)(blockDim.x >> 5) ? s[lane] : Top2{-INFINITY, 0x7fffffff, -INFINITY};
    t = top2_warp(t);
    if (lane == 0) {
        a.part[(size_t)srow * nchunk + chunk] = make_float4(t.v1, __int_as_float(t.i1), t.v2, 0.f);
        __threadfence();
        ticket_s = atomicAdd(a.counters + srow, 1);
    }
    __syncwarp();
    if (ticket_s != nchunk - 1) return;
    __threadfence();
    t = Top2{-INFINITY, 0x7fffffff, -INFINITY};
    for (int c = lane; c < nchunk; c += 32) {
        const float4 p = __ldcg(a.part + (size_t)srow * nchunk + c);
        t = top2_merge(t, Top2{p.x, __float_as_int(p.y), p.z});
    }
    t = top2_warp(t);
    if (lane == 0) {
        a.counters[srow] = 0;
        // a row without any value above -inf (all -inf or NaN) has no maximum: id 0, like a scan that starts at
        // element 0 and never finds anything larger; the id is always a valid row of the embedding table
        const bool none = t.i1 == 0x7fffffff;
        a.tok_out[b * a.Tm + a.tok_col0 + i] = none ? 0 : t.i1;
        if (a.margin_out) a.margin_out[b * a.Tm + i] = none ? 0.f : t.v1 - t.v2;
    }
}

// Greedy acceptance and rollback.  grid = (channel chunks, max(n_rl,1), nb).
//   n = forced_n[b], or the number of leading drafts cand[b][i+1] == g[b][i]
//   committed conv window <- the three raw inputs that end at accepted position n
//   block (0,0,b) also updates the control words: slot, kv_len, pending (= cand[b][0]), outputs.
__global__ void accept_kernel(AcceptArgs a) {
    const int lb = blockIdx.z, b = a.b0 + lb, rl = blockIdx.y;
    const int k = a.k, Tm = a.Tm;
    pdl_trigger();
    pdl_wait();
    const int32_t *cand = a.ctrl.cand + b * Tm, *g = a.ctrl.g + b * Tm;
    int n;
    if (a.forced_n) n = min(max(__ldcg(a.forced_n + b), 0), k);
    else { n = 0; while (n < k && __ldcg(cand + n + 1) == __ldcg(g + n)) ++n; }
    int next = __ldcg(g + n);
    if (a.forced_next && __ldcg(a.forced_next + b) >= 0) next = __ldcg(a.forced_next + b);
    if (next < 0 || next >= a.V) {          // only a caller-supplied id can be out of range: never let it reach the gather
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) atomicCAS(a.ctrl.status, 0, (int)HS_ERR_DEVICE);
        next = 0;
    }
    // conv windows: sequence of raw inputs = [w0 w1 w2 | hist_0 .. hist_k]; new window = entries n+1..n+3
    if (rl < a.n_rl) {
        // the full model's window, then (literal draft state) the draft model's own: the same selection on its buffers
        for (int which = 0; which < (a.dcw ? 2 : 1); ++which) {
            float *cw = (which ? a.dcw : a.cw) + ((size_t)rl * a.B + b) * 3 * a.convd;
            const float *hist = (which ? a.dhist : a.hist) + ((size_t)rl * a.B + b) * Tm * a.convd;
            for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < a.convd; c += gridDim.x * blockDim.x) {
                float v[3];
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    int e = n + 1 + j;
                    v[j] = e < 3 ? __ldcg(cw + e * a.convd + c) : __ldcg(hist + (e - 3) * a.convd + c);
                }
#pragma unroll
                for (int j = 0; j < 3; ++j) cw[j * a.convd + c] = v[j];
            }
        }
    }
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        int32_t *em = a.ctrl.emitted + b * Tm;
        int d[HS_MAX_T];
        for (int i = 0; i < k; ++i) d[i] = __ldcg(cand + i + 1);
        for (int i = 0; i <= k; ++i) em[i] = i < n ? d[i] : (i == n ? next : -1);
        a.ctrl.n_acc[b] = n;
        a.ctrl.slot[b] = a.replay ? 0 : n;
        if (a.dslot) a.dslot[b] = (__ldcg(a.dslot + b) + 1 + n) % a.dslot_mod;
        a.ctrl.kv_len[b] = __ldcg(a.ctrl.kv_len + b) + n + 1;
        a.ctrl.cand[b * Tm] = next;
    }
}

// ------------------------------------------------------------------------------------------------
// Speculative sampling at temperature > 0 (paper Sec. 3.3, Eq. 6).  One block per sequence; a logits row is
// walked in per-thread contiguous segments so that every sum has a fixed order (reproducible draws).
constexpr int SP_THREADS = 1024;

struct RowStat { float mx, Z; };

// max and sum of exp((l - max) / tau) of one row; every thread returns the same values
__device__ __forceinline__ RowStat sp_row_stat(const float *row, int V, float inv_tau, float *red_s) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float mx = -INFINITY;
    for (int j = tid; j < V; j += SP_THREADS) mx = fmaxf(mx, __ldcg(row + j));
    mx = warp_max(mx);
    __syncthreads();
    if (lane == 0) red_s[warp] = mx;
    __syncthreads();
    mx = red_s[0];
    for (int w = 1; w < SP_THREADS / 32; ++w) mx = fmaxf(mx, red_s[w]);
    float z = 0.f;
    for (int j = tid; j < V; j += SP_THREADS) z += expf((__ldcg(row + j) - mx) * inv_tau);
    z = warp_sum(z);
    __syncthreads();
    if (lane == 0) red_s[warp] = z;
    __syncthreads();
    z = 0.f;
    for (int w = 0; w < SP_THREADS / 32; ++w) z += red_s[w];
    return RowStat{mx, z};
}

// Inverse-CDF draw from the unnormalised weights wf(j) >= 0: the smallest j whose cumulative weight exceeds u * total.
// Thread t owns the contiguous segment [t * S, (t + 1) * S); segment sums are scanned in thread order.  Returns the
// index (the same in every thread), or -1 if the total is not positive.
template <class WF>
__device__ __forceinline__ int sp_draw(WF wf, int V, float u, float *seg_s, int *pick_s) {
    const int tid = threadIdx.x;
    const int S = (V + SP_THREADS - 1) / SP_THREADS, j0 = tid * S, j1 = min(V, j0 + S);
    float seg = 0.f;
    for (int j = j0; j < j1; ++j) seg += wf(j);
    __syncthreads();
    seg_s[tid] = seg;
    if (tid == 0) { pick_s[0] = 0x7fffffff; pick_s[1] = 0; }
    __syncthreads();
    // exclusive prefix of this thread's segment and the total: plain ordered sums (1024 adds, once per draw)
    float excl = 0.f, tot = 0.f;
    for (int i = 0; i < SP_THREADS; ++i) { const float v = seg_s[i]; if (i < tid) excl += v; tot += v; }
    if (!(tot > 0.f)) return -1;
    const float t = u * tot;
    if (seg > 0.f && excl + seg > t) atomicMin(pick_s, tid);       // the first segment that reaches past the threshold
    __syncthreads();
    int owner = *pick_s;
    __syncthreads();
    if (owner == 0x7fffffff) {                                     // u * total rounded up to the total: the last positive segment
        if (seg > 0.f) atomicMax(pick_s + 1, tid);
        __syncthreads();
        owner = pick_s[1];
    }
    if (tid == owner) {
        float c = excl; int pick = -1, lastpos = j0;
        for (int j = j0; j < j1; ++j) {
            const float w = wf(j);
            if (w > 0.f) { lastpos = j; c += w; if (c > t) { pick = j; break; } }
        }
        pick_s[2] = pick >= 0 ? pick : lastpos;
    }
    __syncthreads();
    return pick_s[2];
}

struct SampleArgs {
    const float *logits; int64_t row_stride;   // row of sequence b at logits + b * row_stride
    int V, Tm, b0; float inv_tau;
    const float *u; int u_stride, u_col;       // uniform of sequence b at u[b * u_stride + u_col]
    int32_t *tok_out; int tok_col;             // cand[b][tok_col]
};

// draft step: token ~ softmax(logits / tau)
__global__ void __launch_bounds__(SP_THREADS) sample_kernel(const SampleArgs a) {
    __shared__ float red_s[SP_THREADS / 32], seg_s[SP_THREADS];
    __shared__ int pick_s[4];
    const int b = a.b0 + blockIdx.x;
    pdl_trigger();
    pdl_wait();
    const float *row = a.logits + (size_t)b * a.row_stride;
    const RowStat st = sp_row_stat(row, a.V, a.inv_tau, red_s);
    const float u = __ldcg(a.u + (size_t)b * a.u_stride + a.u_col);
    int tok = sp_draw([&](int j) { return expf((__ldcg(row + j) - st.mx) * a.inv_tau); }, a.V, u, seg_s, pick_s);
    if (tok < 0) tok = 0;
    if (threadIdx.x == 0) a.tok_out[b * a.Tm + a.tok_col] = tok;
}

struct SpecAcceptArgs {
    const float *dlogits; int64_t d_seq_stride;     // draft logits: row i of sequence b at dlogits + b * d_seq_stride + i * V
    const float *vlogits;                           // verify logits: row (b - b0) * T + i, V floats each
    const int32_t *cand;                            // [B][Tm]
    const float *u_acc, *u_final; int u_stride;     // u_acc[b * u_stride + i], u_final[b]
    int32_t *n_out, *next_out;                      // [B]: accept length and correction / bonus token
    int V, Tm, k, b0; float inv_tau;
};

// Eq. 6 for one sequence: accept draft i+1 iff u_i < P_H(x) / P_S(x); at the first rejection draw the correction from
// the positive part of P_H - P_S, after k acceptances draw the bonus token from P_H.
__global__ void __launch_bounds__(SP_THREADS) spec_accept_kernel(const SpecAcceptArgs a) {
    __shared__ float red_s[SP_THREADS / 32], seg_s[SP_THREADS];
    __shared__ int pick_s[4];
    const int lb = blockIdx.x, b = a.b0 + lb, T = a.k + 1;
    pdl_trigger();
    pdl_wait();
    const float *drow = a.dlogits + (size_t)b * a.d_seq_stride, *vrow = a.vlogits + (size_t)lb * T * a.V;
    int n = 0;
    RowStat sS{0.f, 1.f}, sH{0.f, 1.f};
    for (; n < a.k; ++n) {
        sS = sp_row_stat(drow + (size_t)n * a.V, a.V, a.inv_tau, red_s);
        sH = sp_row_stat(vrow + (size_t)n * a.V, a.V, a.inv_tau, red_s);
        const int x = __ldcg(a.cand + b * a.Tm + n + 1);
        const float pS = expf((__ldcg(drow + (size_t)n * a.V + x) - sS.mx) * a.inv_tau) / sS.Z;
        const float pH = expf((__ldcg(vrow + (size_t)n * a.V + x) - sH.mx) * a.inv_tau) / sH.Z;
        const float ratio = pS > 0.f ? pH / pS : 1.f;
        if (!(ratio >= 1.f) && !(__ldcg(a.u_acc + (size_t)b * a.u_stride + n) < ratio)) break;      // rejected
    }
    const float uf = __ldcg(a.u_final + b);
    int tok;
    if (n < a.k) {
        const float *dr = drow + (size_t)n * a.V, *vr = vrow + (size_t)n * a.V;
        const float iS = 1.f / sS.Z, iH = 1.f / sH.Z;
        tok = sp_draw([&](int j) {
            const float d = expf((__ldcg(vr + j) - sH.mx) * a.inv_tau) * iH - expf((__ldcg(dr + j) - sS.mx) * a.inv_tau) * iS;
            return d > 0.f ? d : 0.f; }, a.V, uf, seg_s, pick_s);
    } else {
        sH = sp_row_stat(vrow + (size_t)a.k * a.V, a.V, a.inv_tau, red_s);
        tok = -1;
    }
    if (tok < 0) {                                   // bonus draw, or an empty residual: draw from P_H of that position
        const float *vr = vrow + (size_t)n * a.V;
        if (n < a.k) sH = sp_row_stat(vr, a.V, a.inv_tau, red_s);
        tok = sp_draw([&](int j) { return expf((__ldcg(vr + j) - sH.mx) * a.inv_tau); }, a.V, uf, seg_s, pick_s);
        if (tok < 0) tok = 0;
    }
    if (threadIdx.x == 0) { a.n_out[b] = n; a.next_out[b] = tok; }
}

// Self-test of the bounded wait every copy-fed kernel uses: one warp arms an mbarrier for bytes that no copy
// will ever deliver, polls it `polls` times, gives up, records HS_ERR_TIMEOUT and returns.  Nothing is in flight
// when it exits, so the context stays usable.
__global__ void wait_probe_kernel(int32_t *status, int polls) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
    __syncwarp();
    if (threadIdx.x == 0) mbar_expect_tx(&bar, 16);
    __syncwarp();
    const bool ok = __all_sync(0xffffffffu, mbar_wait_n(&bar, 0, polls));
    if (!ok && threadIdx.x == 0) atomicCAS(status, 0, (int)HS_ERR_TIMEOUT);
}

}  // namespace

cudaError_t launch_sample(const float *logits, int64_t row_stride, int V, int Tm, int b0, int nb, float tau,
                          const float *u, int u_stride, int u_col, int32_t *tok_out, int tok_col, cudaStream_t s) {
    SampleArgs a{logits, row_stride, V, Tm, b0, 1.0f / tau, u, u_stride, u_col, tok_out, tok_col};
    return launch_pdl(sample_kernel, dim3(nb), dim3(SP_THREADS), 0, s, a);
}

cudaError_t launch_spec_accept(const float *dlogits, int64_t d_seq_stride, const float *vlogits, const int32_t *cand,
                               const float *u_acc, const float *u_final, int u_stride, int32_t *n_out, int32_t *next_out,
                               int V, int Tm, int k, int b0, int nb, float tau, cudaStream_t s) {
    SpecAcceptArgs a{dlogits, d_seq_stride, vlogits, cand, u_acc, u_final, u_stride, n_out, next_out, V, Tm, k, b0, 1.0f / tau};
    return launch_pdl(spec_accept_kernel, dim3(nb), dim3(SP_THREADS), 0, s, a);
}

cudaError_t launch_wait_probe(int32_t *status, int polls, cudaStream_t s) {
    wait_probe_kernel<<<1, 32, 0, s>>>(status, polls);
    return cudaGetLastError();
}

cudaError_t launch_embed(const __nv_bfloat16 *E, int d, int V, const int32_t *cand, int Tm, int col0, int T,
                         int b0, int nb, float *h, int32_t *status, bool serial, cudaStream_t s) {
    if (serial) {
        // first kernel of a pass: ordinary stream order, so that nothing of this pass (whose kernels read control
        // words in their prologues) starts before everything enqueued earlier - the accept kernel above all - is complete
        embed_kernel<<<dim3(T, nb), dim3(128), 0, s>>>(E, d, V, cand, Tm, col0, T, b0, h, status);
        return cudaGetLastError();
    }
    return launch_pdl(embed_kernel, dim3(T, nb), dim3(128), 0, s, E, d, V, cand, Tm, col0, T, b0, h, status);
}

cudaError_t launch_argmax(const float *logits, int V, int T, int b0, int nb, int Tm,
                          int32_t *tok_out, int tok_col0, float *margin_out, void *part, int32_t *counters, cudaStream_t s) {
    ArgmaxArgs a{logits, V, T, b0, Tm, tok_out, tok_col0, margin_out, reinterpret_cast<float4 *>(part), counters};
    return launch_pdl(argmax_kernel, dim3(HS_ARGMAX_CHUNKS, T, nb), dim3(256), 0, s, a);
}

cudaError_t launch_accept(const AcceptArgs &a, cudaStream_t s) {
    int chunks = (a.convd + 255) / 256;
    if (chunks < 1) chunks = 1;
    return launch_pdl(accept_kernel, dim3(chunks, a.n_rl > 0 ? a.n_rl : 1, a.nb), dim3(256), 0, s, a);
}

// ------------------------------------------------------------------------------------------------
// Argmax without any caller- or library-allocated scratch.
//
// The split argmax above needs a few kilobytes of scratch (per-CTA partial results and a ticket
// counter per row).  Inside the model that scratch is carved out of the caller's work buffer.  This
// stand-alone variant keeps it in a fixed array that is part of the library image instead, so that
// code which is not in a position to allocate device memory can still run the kernel: a host loop
// that already handed every free byte of the GPU to its own arena, a plug-in that is only given
// pointers, or a latency-critical section where an allocation (which may synchronise the device)
// is not acceptable.  The price: the array is loaded on every GPU that loads the library and stays
// until the process exits, and all calls share it.
constexpr int HS_STATIC_ROWS = 64;         // most logits rows one call may pass
constexpr size_t HS_STATIC_PART_BYTES = (size_t)HS_STATIC_ROWS * HS_ARGMAX_CHUNKS * 16;
constexpr size_t HS_STATIC_BYTES = HS_STATIC_PART_BYTES + HS_STATIC_ROWS * 4;   // partials, then counters: 33 KB
static __device__ __align__(256) unsigned char hs_static_scratch[HS_STATIC_BYTES];

namespace {
constexpr int HS_STATIC_MAX_DEVICES = 64;
void *g_static_ptr[HS_STATIC_MAX_DEVICES];     // device address of hs_static_scratch, per device; null = not looked up yet
std::mutex g_static_mutex;                     // two host threads may make their first call at the same time
}

extern "C" int hs_argmax_static(const float *logits_dev, int V, int rows, int32_t *token_dev, float *margin_dev, void *stream) {
    if (!logits_dev || !token_dev || V < 1 || rows < 1) return HS_ERR_INVALID_ARG;
    if (rows > HS_STATIC_ROWS) return HS_ERR_SIZE;             // more rows than the built-in scratch holds
    // the kernel reads rows of a width that is a multiple of four with 128-bit loads: such rows must start on a
    // 16-byte boundary (a view that begins inside a larger tensor may not); the outputs are plain 32-bit words
    if (((uintptr_t)logits_dev & ((V & 3) == 0 ? 15u : 3u)) || ((uintptr_t)token_dev & 3u) || ((uintptr_t)margin_dev & 3u))
        return HS_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= HS_STATIC_MAX_DEVICES) return HS_ERR_CUDA;
    unsigned char *base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            // In host code the array's name is only a handle; the address a kernel can use has to be asked for,
            // once per device, with that device current.
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, hs_static_scratch) != cudaSuccess || !p) return HS_ERR_CUDA;
            g_static_ptr[dev] = p;
        }
        base = static_cast<unsigned char *>(g_static_ptr[dev]);
    }
    int32_t *counters = reinterpret_cast<int32_t *>(base + HS_STATIC_PART_BYTES);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the tickets must start at zero whatever an earlier (possibly failed) call left behind
    if (cudaMemsetAsync(counters, 0, (size_t)rows * 4, s) != cudaSuccess) return HS_ERR_CUDA;
    ArgmaxArgs a{logits_dev, V, rows, 0, rows, token_dev, 0, margin_dev, reinterpret_cast<float4 *>(base), counters};
    argmax_kernel<<<dim3(HS_ARGMAX_CHUNKS, rows, 1), 256, 0, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? HS_OK : HS_ERR_CUDA;
}

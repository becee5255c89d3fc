// Skinny projection kernel (CUDA cores): out[r][o] = sum_j W[o][j] * x[r][j] for a handful of
// activation rows r (batch * (k+1) <= 16), bf16 weights streamed exactly once from HBM, fp32
// activations and accumulation.  Every weight byte is used only `rows` times, so the kernel is
// HBM-bound and its job is to keep the weight stream running through the dependency stalls of a
// decode step:
//
//  * The weight matrix is cut into one tile per CTA - a contiguous range of output rows times a
//    range of the reduction dimension (a "K split"; only the residual epilogue may split K, its
//    partial sums are written as separate parts that the consumer adds in a fixed order, so the
//    result is bit-reproducible and needs no atomics).  grid = one CTA per SM.
//  * A CTA streams its tile through a ring of shared-memory stages filled by bulk asynchronous
//    copies (one per weight row, completion counted on an mbarrier).  The first stages are issued
//    BEFORE the programmatic-dependent-launch wait: they depend on nothing the previous kernel
//    computes, so the next kernel's weights are already on their way into shared memory while the
//    current kernel is still running.
//  * After the wait the activation rows are staged in shared memory (summing the parts of the
//    producer, with the optional RMSNorm weight folded in; the 1/rms factor is a per-row scalar and
//    is applied in the epilogue), and 8 warps consume the stages: a warp owns 8 weight rows and an
//    interleaved set of 256-column blocks, keeps 8*R accumulators, and reduces them with one
//    transposing shuffle reduction.
// Epilogues: plain store, residual add (with K split), SwiGLU over interleaved gate/up rows.
#include "hs_internal.h"
#include "hs_device.cuh"
#include <cstdio>
#include <cstdlib>

namespace {
using namespace hsd;

constexpr int GV_WARPS = 8;
constexpr int GV_THREADS = GV_WARPS * 32;
constexpr int GV_MAXROWS = 16;      // activation rows per launch
constexpr int GV_MAXDEPTH = 4;

struct GemvGeo {
    int S0, S1;          // K splits of segment 0 / 1
    int kr0, kr1;        // nominal K-range width per split (multiple of 256; the last may be shorter)
    int NR;              // row ranges; grid = NR * (S0 + S1)
    int unit;            // row ranges start on multiples of this (2 for the SwiGLU epilogue)
    int kc;              // columns per tile (multiple of 256): a K range is walked in chunks of kc
    int D;               // tiles in flight per warp (depth of each warp's private ring)
    int krmax;           // max(kr0, kr1): row stride of the staged activations
    int off_x, off_nw, off_ring; // shared-memory carve-up (bytes)
    int rq, rrem;        // row ranges: units / NR and units % NR
    int nch;             // chunks of a full K range
    long long pf_per;    // bytes of the next projection's weights each CTA pulls into L2
    int cl, off_part;    // cl = 1: the K splits of a row range form a thread-block cluster and reduce their partial sums
                         // through distributed shared memory (one part out); off_part: [rows of the range][16] floats
};

// Residual epilogue with the K split reduced inside the cluster.  Every CTA has left the partial sums of its K
// range in part_s[local output row][activation row]; the S CTAs of the cluster (rank = K split index) share the
// row range.  Rank q finishes a contiguous share of the rows: partials added in rank order, then the residual -
// a fixed order, so the result does not depend on timing.  The second barrier keeps every CTA's shared memory
// alive until its peers have read it.
template <int THREADS>
__device__ __forceinline__ void cluster_reduce_resid(const GemvArgs &a, float *part_s, int S, int q, int r0, int nrow, int nrows) {
    __syncthreads();
    cluster_arrive(); cluster_wait();
    const int lo = nrow * q / S, nloc = nrow * (q + 1) / S - lo;
#pragma unroll 1
    for (int idx = threadIdx.x; idx < nloc * nrows; idx += THREADS) {
        const int xr = idx / nloc, row = lo + idx - xr * nloc;            // consecutive threads: consecutive outputs
        const size_t oi = (size_t)xr * a.ldo + r0 + row;
        float res[HS_H_PARTS];
#pragma unroll
        for (int p = 0; p < HS_H_PARTS; ++p) res[p] = p < a.rparts ? __ldcg(a.resid + (size_t)p * a.rpstride + oi) : 0.f;
        const uint32_t local = smem_u32(part_s + row * GV_MAXROWS + xr);
        float v[HS_H_PARTS];
#pragma unroll
        for (int p = 0; p < HS_H_PARTS; ++p) v[p] = p < S ? dsmem_ld_f32(dsmem_addr(local, (uint32_t)p)) : 0.f;
        float sum = v[0];
#pragma unroll
        for (int p = 1; p < HS_H_PARTS; ++p) sum += v[p];
#pragma unroll
        for (int p = 0; p < HS_H_PARTS; ++p) sum += res[p];
        a.out[oi] = sum;
    }
    cluster_arrive(); cluster_wait();
}

__device__ __forceinline__ float dot8(const uint4 &w, const float4 &a, const float4 &b, float acc) {
    acc = fmaf(bf_lo(w.x), a.x, acc); acc = fmaf(bf_hi(w.x), a.y, acc);
    acc = fmaf(bf_lo(w.y), a.z, acc); acc = fmaf(bf_hi(w.y), a.w, acc);
    acc = fmaf(bf_lo(w.z), b.x, acc); acc = fmaf(bf_hi(w.z), b.y, acc);
    acc = fmaf(bf_lo(w.w), b.z, acc); acc = fmaf(bf_hi(w.w), b.w, acc);
    return acc;
}

// Position of activation column c (a multiple of 4) inside its staged row.  Within every block of 256
// columns the lane that owns columns 8l..8l+7 finds its first four floats at 4l and the next four at
// 128 + 4l, so that both 128-bit reads of a warp are contiguous (no bank conflicts).
__device__ __forceinline__ int xs_pos(int c) {
    const int within = c & 255;
    return (c & ~255) + ((within >> 2) & 1) * 128 + (within >> 3) * 4;
}

// R activation rows per pass in registers, WR weight rows per warp tile.
// A tile is WR weight rows x kc columns; warp w owns the row groups w, w + 8, ... of the CTA's row
// range and walks each group's K chunks in order through a private ring of D tile buffers, so the
// main loop needs no block-wide synchronisation.
// ONE = true is the lean instance for exactly R activation rows (1: the draft step, 2 or 3: verify at k = 1, 2)
// with the epilogue (EPI) and the presence of a norm (NORMED) fixed at compile time: the same program with every
// unused path removed.  A step is a chain of ~3 us kernels, so the length of the executed code is a first-order
// cost there.  ONE = false (EPI = NORMED = -1: taken from the arguments) is the general form.
// SEG = false: the instance knows there is no second weight segment.
template <int R, int WR, bool ONE = false, int EPI = -1, int NORMED = -1, bool SEG = true>
__global__ void __launch_bounds__(GV_THREADS, 2) gemv_kernel(const GemvArgs a, const GemvGeo g, int32_t *status) {
    static_assert(WR * R <= 32, "a warp reduces at most 32 values");
    constexpr int NV = pow2_ge(WR * R);
    constexpr int LPV = 32 / NV;
    extern __shared__ __align__(128) unsigned char smraw[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smraw);                 // [8][D]
    float *rstd_s = reinterpret_cast<float *>(smraw + 256);               // [16]
    float *ss_s = rstd_s + GV_MAXROWS;                                    // [8][16]
    float *x_s = reinterpret_cast<float *>(smraw + g.off_x);              // [nrows][krmax]
    float *nw_s = reinterpret_cast<float *>(smraw + g.off_nw);            // [krmax] norm weights of this K range
    __nv_bfloat16 *ring = reinterpret_cast<__nv_bfloat16 *>(smraw + g.off_ring);   // [8][D][WR][kc]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int si = blockIdx.x, ri = blockIdx.y;          // grid = (K splits, row ranges): no division to find them
    const bool seg1 = SEG ? si >= g.S0 : false;
    const __nv_bfloat16 *W = seg1 ? a.W1 : a.W0;
    const int ld = seg1 ? a.ldw1 : a.ldw0, Kseg = seg1 ? a.K1 : a.K0;
    const int krn = seg1 ? g.kr1 : g.kr0;
    const int k0 = (seg1 ? si - g.S0 : si) * krn;
    const int kr = min(krn, Kseg - k0);
    // row ranges: the first g.rrem ranges have g.rq + 1 units, the others g.rq (computed once on the host)
    const int r0 = (ri * g.rq + min(ri, g.rrem)) * g.unit;
    const int nrow = (g.rq + (ri < g.rrem ? 1 : 0)) * g.unit, r1 = r0 + nrow;
    const int kc = g.kc, D = g.D, krmax = g.krmax;
    int nch = g.nch;                                      // chunks of a full K range; the last range may need fewer
    while ((nch - 1) * kc >= kr) --nch;
    const int ngrp = (nrow + WR - 1) / WR;
    const int mygrps = warp < ngrp ? (ngrp - warp + GV_WARPS - 1) / GV_WARPS : 0;
    const int ntile = mygrps * nch;
    uint64_t *mybar = bars + warp * D;
    __nv_bfloat16 *mybuf = ring + (size_t)warp * D * WR * kc;

    // tiles are requested strictly in order: (group, chunk, buffer) of the next request advance as counters
    int i_gi = 0, i_ch = 0, i_buf = 0;
    auto issue_tile = [&]() {              // whole warp
        const int gi = i_gi, ch = i_ch, buf = i_buf;
        if (++i_ch == nch) { i_ch = 0; ++i_gi; }
        if (++i_buf == D) i_buf = 0;
        const int row0 = r0 + (warp + gi * GV_WARPS) * WR;
        const int rows_in = min(WR, r1 - row0);
        const int cw = min(kc, kr - ch * kc);
        if (lane == 0) mbar_expect_tx(&mybar[buf], (uint32_t)rows_in * cw * 2);
        __syncwarp();
        if (ld == kc && cw == kc) {
            // whole rows of an unsplit matrix: the tile is one contiguous piece of memory, one large request
            if (lane == 0)
                bulk_g2s(mybuf + (size_t)buf * WR * kc, W + (size_t)row0 * ld, (uint32_t)rows_in * cw * 2, &mybar[buf]);
        } else if (lane < rows_in) {
            bulk_g2s(mybuf + ((size_t)buf * WR + lane) * kc, W + (size_t)(row0 + lane) * ld + k0 + ch * kc,
                     (uint32_t)cw * 2, &mybar[buf]);
        }
    };

    // ---- prologue, independent of the previous kernel: start the weight stream
    if (a.early_trigger) pdl_trigger();
    if (tid < GV_WARPS * D) { mbar_init(&bars[tid], 1); mbar_fence_init(); }
    __syncthreads();
    {
        const int pre = min(D, ntile);
#pragma unroll 1
        for (int t = 0; t < pre; ++t) issue_tile();
    }
    // pull the next projection's weights towards L2: by the time its own kernel asks for them the
    // HBM latency is already paid
    if (a.pf_bytes > 0 && warp == GV_WARPS - 1) {
        const long long per = g.pf_per;                   // bytes per CTA, a multiple of 16
        const long long lo = (long long)(ri * gridDim.x + si) * per, hi = min(lo + per, (long long)a.pf_bytes & ~15ll);
#pragma unroll 1
        for (long long o = lo + (long long)lane * 8192; o < hi; o += 32 * 8192)
            prefetch_l2(reinterpret_cast<const char *>(a.pf_ptr) + o, (uint32_t)min(8192ll, hi - o));
    }
    // the norm weights are parameters too: fetch them now, they would otherwise miss in L2 after the wait
    const bool normed = NORMED >= 0 ? (NORMED != 0 && !seg1) : (a.norm_w != nullptr && !seg1);
    const int epi = EPI >= 0 ? EPI : a.epi;
    if (normed)
#pragma unroll 1
        for (int c = tid * 4; c < kr; c += GV_THREADS * 4)
            *reinterpret_cast<float4 *>(nw_s + c) = *reinterpret_cast<const float4 *>(a.norm_w + k0 + c);
    pdl_wait();
    if (!a.early_trigger) pdl_trigger();
    __syncthreads();                       // nw_s complete

    // ---- stage the activation rows of this K range (parts summed, norm weight folded in)
    const int nrows = ONE ? R : a.nrows;
    {
        const float *xsrc = seg1 ? a.x1 : a.x0;
        const int ldx = seg1 ? a.ldx1 : a.ldx0;
        const int parts = seg1 ? 1 : a.xparts;
        const int c_lo = normed ? 0 : k0, c_hi = normed ? Kseg : k0 + kr;
        constexpr int SR = ONE ? R : 4;                     // activation rows staged per sweep
#pragma unroll 1
        for (int rbase = 0; rbase < nrows; rbase += SR) {
            float ss[SR];
#pragma unroll
            for (int j = 0; j < SR; ++j) ss[j] = 0.f;
#pragma unroll 1
            for (int c = c_lo + tid * 4; c < c_hi; c += GV_THREADS * 4) {
                float4 v[SR];
#pragma unroll
                for (int j = 0; j < SR; ++j) {             // all loads of the rows of a sweep are in flight together
                    v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (rbase + j < nrows) {
                        const float *p = xsrc + (size_t)(rbase + j) * ldx + c;
                        v[j] = __ldcg(reinterpret_cast<const float4 *>(p));
                        float4 u[HS_H_PARTS - 1];           // all parts in flight together, added in order
#pragma unroll
                        for (int q = 1; q < HS_H_PARTS; ++q)
                            if (q < parts) u[q - 1] = __ldcg(reinterpret_cast<const float4 *>(p + (size_t)q * a.xpstride));
#pragma unroll
                        for (int q = 1; q < HS_H_PARTS; ++q)
                            if (q < parts) { v[j].x += u[q - 1].x; v[j].y += u[q - 1].y; v[j].z += u[q - 1].z; v[j].w += u[q - 1].w; }
                    }
                }
                const bool inside = c >= k0 && c < k0 + kr;
                float4 nw = make_float4(1.f, 1.f, 1.f, 1.f);
                if (normed && inside) nw = *reinterpret_cast<const float4 *>(nw_s + (c - k0));
#pragma unroll
                for (int j = 0; j < SR; ++j) {
                    if (rbase + j >= nrows) continue;
                    ss[j] = fmaf(v[j].x, v[j].x, fmaf(v[j].y, v[j].y, fmaf(v[j].z, v[j].z, fmaf(v[j].w, v[j].w, ss[j]))));
                    if (inside)
                        *reinterpret_cast<float4 *>(x_s + (size_t)(rbase + j) * krmax + xs_pos(c - k0)) =
                            make_float4(v[j].x * nw.x, v[j].y * nw.y, v[j].z * nw.z, v[j].w * nw.w);
                }
            }
            if (normed) {
#pragma unroll
                for (int j = 0; j < SR; ++j) {
                    const float t = warp_sum(ss[j]);
                    if (lane == 0 && rbase + j < nrows) ss_s[warp * GV_MAXROWS + rbase + j] = t;
                }
            }
        }
    }
    __syncthreads();

    // which result this lane holds after the transposing reduction: value v = (r, w)
    const int vidx = lane / LPV, vr = vidx / WR, vw = vidx - vr * WR;
    const bool holder = (lane & (LPV - 1)) == 0 && vidx < WR * R;
    bool bad = false;
    int g_buf = 0; uint32_t g_phase = 0;   // buffer and barrier phase of the first tile of the current row group
    int t_next = min(D, ntile);            // tiles requested so far
#pragma unroll 1
    for (int gi = 0; gi < mygrps; ++gi) {
        const int row0 = r0 + (warp + gi * GV_WARPS) * WR;
        const int rows_in = min(WR, r1 - row0);
        int c_buf = g_buf; uint32_t c_phase = g_phase;
#pragma unroll 1
        for (int p0 = 0; p0 < nrows; p0 += R) {
            c_buf = g_buf; c_phase = g_phase;               // every pass walks the group's tiles from its first buffer
            // residual of the value this lane will own: in flight while the tile is reduced
            float res = 0.f;
            const bool live = holder && p0 + vr < nrows && vw < rows_in;
            const size_t oi = (size_t)(p0 + vr) * a.ldo + row0 + vw;
            if (epi == EPI_RESID && si == 0 && live)
            {
                float rq[HS_H_PARTS];
#pragma unroll
                for (int q = 0; q < HS_H_PARTS; ++q) rq[q] = q < a.rparts ? __ldcg(a.resid + (size_t)q * a.rpstride + oi) : 0.f;
#pragma unroll
                for (int q = 0; q < HS_H_PARTS; ++q) res += rq[q];
            }
            float acc[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) acc[i] = 0.f;
#pragma unroll 1
            for (int ch = 0; ch < nch; ++ch) {
                const int buf = c_buf;
                if (p0 == 0 && !__all_sync(0xffffffffu, mbar_wait(&mybar[buf], c_phase))) { bad = true; break; }
                const __nv_bfloat16 *tile = mybuf + (size_t)buf * WR * kc;
                const int nb = min(kc, kr - ch * kc) >> 8;
#pragma unroll 2
                for (int blk = 0; blk < nb; ++blk) {
                    const int col = (blk << 8) + lane * 8;
                    uint4 wv[WR];
#pragma unroll
                    for (int w = 0; w < WR; ++w) wv[w] = *reinterpret_cast<const uint4 *>(tile + (size_t)w * kc + col);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const float *xr = x_s + (size_t)min(p0 + r, nrows - 1) * krmax + ch * kc + (blk << 8) + lane * 4;
                        const float4 xa = *reinterpret_cast<const float4 *>(xr);
                        const float4 xb = *reinterpret_cast<const float4 *>(xr + 128);
#pragma unroll
                        for (int w = 0; w < WR; ++w) acc[r * WR + w] = dot8(wv[w], xa, xb, acc[r * WR + w]);
                    }
                }
                // last pass over the activation rows: this buffer is free, refill it D tiles ahead
                if (p0 + R >= nrows) {
                    __syncwarp();
                    if (t_next < ntile) { issue_tile(); ++t_next; }
                }
                if (++c_buf == D) { c_buf = 0; c_phase ^= 1u; }
            }
            if (bad) break;
            float tot = xreduce<NV>(acc, lane);
            if (normed) {
                float t = 0.f;
#pragma unroll
                for (int w = 0; w < GV_WARPS; ++w) t += ss_s[w * GV_MAXROWS + min(p0 + vr, nrows - 1)];
                tot *= rsqrtf(t / (float)Kseg + a.eps);
            }
            if (epi == EPI_SWIGLU) {
                const float up = __shfl_down_sync(0xffffffffu, tot, LPV);    // value v + 1 = the up row of the pair
                if (live && !(vw & 1)) a.out[(size_t)(p0 + vr) * a.ldo + ((row0 + vw) >> 1)] = silu_f(tot) * up;
            } else if (live) {
                if (epi == EPI_RESID) a.out[(size_t)si * a.opstride + oi] = tot + res;
                else a.out[oi] = tot;
            }
        }
        if (bad) break;
        g_buf = c_buf; g_phase = c_phase;
    }
    if (bad) atomicCAS(status, 0, (int)HS_ERR_TIMEOUT);     // a copy never landed
}

// ------------------------------------------------------------------------------------------------
// Tensor-core variant for 2..16 activation rows (verify passes, small batches).  Same tiling, ring and
// prologue as above; the inner product runs on mma.sync m16n8k16 with the roles swapped to fit the
// shapes: the M = 16 rows of the A operand are 8 activation rows as bf16 head (rows 0-7) and bf16
// remainder (rows 8-15) - so the fp32 activations enter exactly to 2^-17 - and the N = 8 columns are
// the 8 weight rows of a warp's tile, read straight from the streamed bf16 tile (rows padded by 16
// bytes so that ldmatrix is conflict-free).  Four accumulators per row group take the k steps in turn,
// which keeps the MMA pipeline full.  NG = groups of 8 activation rows (1 or 2).
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// EPI / NORMED >= 0 fix the epilogue and the presence of a norm at compile time (shorter program, see above).
// CL: residual epilogue with the K split reduced inside a thread-block cluster (cluster_reduce_resid).
template <int NG, int EPI = -1, int NORMED = -1, bool CL = false>
__global__ void __launch_bounds__(GV_THREADS, 2) gemm_mma_kernel(const GemvArgs a, const GemvGeo g, int32_t *status) {
    constexpr int WR = 8;
    extern __shared__ __align__(128) unsigned char smraw[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smraw);                 // [8][D]
    float *ss_s = reinterpret_cast<float *>(smraw + 256);                 // [8][16]
    __nv_bfloat16 *xa_s = reinterpret_cast<__nv_bfloat16 *>(smraw + g.off_x);      // [NG][16][KP]
    float *nw_s = reinterpret_cast<float *>(smraw + g.off_nw);            // [krmax]
    __nv_bfloat16 *ring = reinterpret_cast<__nv_bfloat16 *>(smraw + g.off_ring);   // [8][D][WR][kc + 8]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int si = blockIdx.x, ri = blockIdx.y;          // grid = (K splits, row ranges)
    const bool seg1 = si >= g.S0;
    const __nv_bfloat16 *W = seg1 ? a.W1 : a.W0;
    const int ld = seg1 ? a.ldw1 : a.ldw0, Kseg = seg1 ? a.K1 : a.K0;
    const int krn = seg1 ? g.kr1 : g.kr0;
    const int k0 = (seg1 ? si - g.S0 : si) * krn;
    const int kr = min(krn, Kseg - k0);
    const int r0 = (ri * g.rq + min(ri, g.rrem)) * g.unit;
    const int nrow = (g.rq + (ri < g.rrem ? 1 : 0)) * g.unit, r1 = r0 + nrow;
    const int kc = g.kc, D = g.D, krmax = g.krmax, TS = kc + 8, KP = krmax + 8;
    int nch = g.nch;                                      // chunks of a full K range; the last range may need fewer
    while ((nch - 1) * kc >= kr) --nch;
    const int ngrp = (nrow + WR - 1) / WR;
    const int mygrps = warp < ngrp ? (ngrp - warp + GV_WARPS - 1) / GV_WARPS : 0;
    const int ntile = mygrps * nch;
    uint64_t *mybar = bars + warp * D;
    __nv_bfloat16 *mybuf = ring + (size_t)warp * D * WR * TS;

    int i_gi = 0, i_ch = 0, i_buf = 0;     // (group, chunk, buffer) of the next request
    auto issue_tile = [&]() {              // whole warp
        const int gi = i_gi, ch = i_ch, buf = i_buf;
        if (++i_ch == nch) { i_ch = 0; ++i_gi; }
        if (++i_buf == D) i_buf = 0;
        const int row0 = r0 + (warp + gi * GV_WARPS) * WR;
        const int rows_in = min(WR, r1 - row0);
        const int cw = min(kc, kr - ch * kc);
        if (lane == 0) mbar_expect_tx(&mybar[buf], (uint32_t)rows_in * cw * 2);
        __syncwarp();
        if (lane < rows_in)
            bulk_g2s(mybuf + ((size_t)buf * WR + lane) * TS, W + (size_t)(row0 + lane) * ld + k0 + ch * kc,
                     (uint32_t)cw * 2, &mybar[buf]);
    };

    // ---- prologue, independent of the previous kernel
    if (a.early_trigger) pdl_trigger();
    if (tid < GV_WARPS * D) { mbar_init(&bars[tid], 1); mbar_fence_init(); }
    __syncthreads();
    {
        const int pre = min(D, ntile);
#pragma unroll 1
        for (int t = 0; t < pre; ++t) issue_tile();
    }
    if (a.pf_bytes > 0 && warp == GV_WARPS - 1) {
        const long long per = g.pf_per;
        const long long lo = (long long)(ri * gridDim.x + si) * per, hi = min(lo + per, (long long)a.pf_bytes & ~15ll);
#pragma unroll 1
        for (long long o = lo + (long long)lane * 8192; o < hi; o += 32 * 8192)
            prefetch_l2(reinterpret_cast<const char *>(a.pf_ptr) + o, (uint32_t)min(8192ll, hi - o));
    }
    const bool normed = NORMED >= 0 ? (NORMED != 0 && !seg1) : (a.norm_w != nullptr && !seg1);
    const int epi = EPI >= 0 ? EPI : a.epi;
    if (normed)
#pragma unroll 1
        for (int c = tid * 4; c < kr; c += GV_THREADS * 4)
            *reinterpret_cast<float4 *>(nw_s + c) = *reinterpret_cast<const float4 *>(a.norm_w + k0 + c);
    const int nrows = a.nrows;
    // activation rows that do not exist are zero in both halves of their group
#pragma unroll 1
    for (int r = nrows; r < NG * 8; ++r) {
        __nv_bfloat16 *p = xa_s + ((size_t)(r >> 3) * 16 + (r & 7)) * KP;
#pragma unroll 1
        for (int c = tid * 8; c < kr; c += GV_THREADS * 8) {
            *reinterpret_cast<uint4 *>(p + c) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4 *>(p + 8 * KP + c) = make_uint4(0, 0, 0, 0);
        }
    }
    pdl_wait();
    if (!a.early_trigger) pdl_trigger();
    __syncthreads();                       // nw_s complete

    // ---- stage the activation rows of this K range as bf16 head + remainder (parts summed, norm weight folded in)
    {
        const float *xsrc = seg1 ? a.x1 : a.x0;
        const int ldx = seg1 ? a.ldx1 : a.ldx0;
        const int parts = seg1 ? 1 : a.xparts;
        const int c_lo = normed ? 0 : k0, c_hi = normed ? Kseg : k0 + kr;
        constexpr int SR = 5;               // rows per sweep: k = 4 (five rows) is staged in one trip to L2
#pragma unroll 1
        for (int rbase = 0; rbase < nrows; rbase += SR) {
            float ss[SR];
#pragma unroll
            for (int j = 0; j < SR; ++j) ss[j] = 0.f;
            for (int c = c_lo + tid * 4; c < c_hi; c += GV_THREADS * 4) {
                float4 v[SR];
#pragma unroll
                for (int j = 0; j < SR; ++j) {             // all loads of the rows of a sweep are in flight together
                    v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (rbase + j < nrows) {
                        const float *p = xsrc + (size_t)(rbase + j) * ldx + c;
                        v[j] = __ldcg(reinterpret_cast<const float4 *>(p));
                        float4 u[HS_H_PARTS - 1];           // all parts in flight together, added in order
#pragma unroll
                        for (int q = 1; q < HS_H_PARTS; ++q)
                            if (q < parts) u[q - 1] = __ldcg(reinterpret_cast<const float4 *>(p + (size_t)q * a.xpstride));
#pragma unroll
                        for (int q = 1; q < HS_H_PARTS; ++q)
                            if (q < parts) { v[j].x += u[q - 1].x; v[j].y += u[q - 1].y; v[j].z += u[q - 1].z; v[j].w += u[q - 1].w; }
                    }
                }
                const bool inside = c >= k0 && c < k0 + kr;
                float4 nw = make_float4(1.f, 1.f, 1.f, 1.f);
                if (normed && inside) nw = *reinterpret_cast<const float4 *>(nw_s + (c - k0));
#pragma unroll
                for (int j = 0; j < SR; ++j) {
                    const int r = rbase + j;
                    if (r >= nrows) continue;
                    ss[j] = fmaf(v[j].x, v[j].x, fmaf(v[j].y, v[j].y, fmaf(v[j].z, v[j].z, fmaf(v[j].w, v[j].w, ss[j]))));
                    if (inside) {
                        const float x[4] = {v[j].x * nw.x, v[j].y * nw.y, v[j].z * nw.z, v[j].w * nw.w};
                        __nv_bfloat16 h[4], l[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) { h[e] = __float2bfloat16_rn(x[e]); l[e] = __float2bfloat16_rn(x[e] - __bfloat162float(h[e])); }
                        __nv_bfloat16 *p = xa_s + ((size_t)(r >> 3) * 16 + (r & 7)) * KP + (c - k0);
                        *reinterpret_cast<uint2 *>(p) = make_uint2((uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16),
                                                                   (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16));
                        *reinterpret_cast<uint2 *>(p + 8 * KP) = make_uint2((uint32_t)__bfloat16_as_ushort(l[0]) | ((uint32_t)__bfloat16_as_ushort(l[1]) << 16),
                                                                            (uint32_t)__bfloat16_as_ushort(l[2]) | ((uint32_t)__bfloat16_as_ushort(l[3]) << 16));
                    }
                }
            }
            if (normed) {
#pragma unroll
                for (int j = 0; j < SR; ++j) {
                    const float t = warp_sum(ss[j]);
                    if (lane == 0 && rbase + j < nrows) ss_s[warp * GV_MAXROWS + rbase + j] = t;
                }
            }
        }
    }
    __syncthreads();

    // this lane's results: activation row g * 8 + g8, weight rows 2 * t4 and 2 * t4 + 1 of the tile
    const int g8 = lane >> 2, t4 = lane & 3;
    bool bad = false;
    int c_buf = 0; uint32_t c_phase = 0;   // buffer and barrier phase of the next tile to consume
    int t_next = min(D, ntile);            // tiles requested so far
#pragma unroll 1
    for (int gi = 0; gi < mygrps && !bad; ++gi) {
        const int row0 = r0 + (warp + gi * GV_WARPS) * WR;
        const int rows_in = min(WR, r1 - row0);
        const int wrow = row0 + 2 * t4;
        float res[NG][2];
#pragma unroll
        for (int gq = 0; gq < NG; ++gq) {
            res[gq][0] = res[gq][1] = 0.f;
            const int xr = gq * 8 + g8;
            if (!CL && epi == EPI_RESID && si == 0 && xr < nrows)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (2 * t4 + e < rows_in)
                        for (int q = 0; q < a.rparts; ++q) res[gq][e] += __ldcg(a.resid + (size_t)q * a.rpstride + (size_t)xr * a.ldo + wrow + e);
        }
        float acc[NG][4][4];
#pragma unroll
        for (int gq = 0; gq < NG; ++gq)
#pragma unroll
            for (int j = 0; j < 4; ++j) { acc[gq][j][0] = acc[gq][j][1] = acc[gq][j][2] = acc[gq][j][3] = 0.f; }
#pragma unroll 1
        for (int ch = 0; ch < nch; ++ch) {
            const int buf = c_buf;
            if (!__all_sync(0xffffffffu, mbar_wait(&mybar[buf], c_phase))) { bad = true; break; }
            const __nv_bfloat16 *tile = mybuf + (size_t)buf * WR * TS;
            const int cw = min(kc, kr - ch * kc);
            const __nv_bfloat16 *brow = tile + (size_t)(lane & 7) * TS + (lane >> 3) * 8;
            const __nv_bfloat16 *arow = xa_s + (size_t)((lane & 7) + ((lane >> 3) & 1) * 8) * KP + ch * kc + (lane >> 4) * 8;
            for (int kk = 0; kk < cw; kk += 64) {              // four k steps per round, one accumulator each
                uint32_t bw[2][4];
                ldsm_x4(bw[0], brow + kk);
                ldsm_x4(bw[1], brow + kk + 32);
#pragma unroll
                for (int gq = 0; gq < NG; ++gq)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t af[4];
                        ldsm_x4(af, arow + (size_t)gq * 16 * KP + kk + j * 16);
                        mma_bf16(acc[gq][j], af, bw[j >> 1][(j & 1) * 2], bw[j >> 1][(j & 1) * 2 + 1]);
                    }
            }
            __syncwarp();
            if (t_next < ntile) { issue_tile(); ++t_next; }     // this buffer is free: refill it D tiles ahead
            if (++c_buf == D) { c_buf = 0; c_phase ^= 1u; }
        }
        if (bad) break;
#pragma unroll
        for (int gq = 0; gq < NG; ++gq) {
            const int xr = gq * 8 + g8;
            float v[2];
#pragma unroll
            for (int e = 0; e < 2; ++e)                           // head rows (c0, c1) + remainder rows (c2, c3), four partial sums
                v[e] = (acc[gq][0][e] + acc[gq][1][e]) + (acc[gq][2][e] + acc[gq][3][e]) +
                       ((acc[gq][0][2 + e] + acc[gq][1][2 + e]) + (acc[gq][2][2 + e] + acc[gq][3][2 + e]));
            if (normed) {
                float t = 0.f;
#pragma unroll
                for (int w = 0; w < GV_WARPS; ++w) t += ss_s[w * GV_MAXROWS + min(xr, nrows - 1)];
                const float rs = rsqrtf(t / (float)Kseg + a.eps);
                v[0] *= rs; v[1] *= rs;
            }
            if (xr >= nrows) continue;
            if (epi == EPI_SWIGLU) {
                if (2 * t4 + 1 < rows_in) a.out[(size_t)xr * a.ldo + (wrow >> 1)] = silu_f(v[0]) * v[1];
            } else {
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (2 * t4 + e < rows_in) {
                        const size_t oi = (size_t)xr * a.ldo + wrow + e;
                        if (CL) reinterpret_cast<float *>(smraw + g.off_part)[(wrow + e - r0) * GV_MAXROWS + xr] = v[e];
                        else if (epi == EPI_RESID) a.out[(size_t)si * a.opstride + oi] = v[e] + res[gq][e];
                        else a.out[oi] = v[e];
                    }
            }
        }
    }
    if (CL) cluster_reduce_resid<GV_THREADS>(a, reinterpret_cast<float *>(smraw + g.off_part), (int)gridDim.x, si, r0, nrow, nrows);
    if (bad) atomicCAS(status, 0, (int)HS_ERR_TIMEOUT);     // a copy never landed
}

int g_sms = 148;
int g_max_clusters[HS_H_PARTS + 1] = {0, 0, 0, 0, 0};   // resident clusters by cluster size (0: clusters unavailable)
}  // namespace
bool g_hs_gemm_mma = true;
bool g_hs_cluster_reduce = true;   // residual projections of 4..16 rows reduce their K split inside a thread-block cluster
namespace {
constexpr size_t GV_SMEM_MAX = 224 * 1024;
constexpr size_t GV_SMEM_PAIR = 127 * 1024;   // below this the CTA of the next kernel fits beside it

template <int NG>
cudaError_t launch_mma(const GemvArgs &a, const GemvGeo &g, size_t smem, int32_t *status, cudaStream_t s) {
    const dim3 grid(g.S0 + g.S1, g.NR), block(GV_THREADS);
    const int nm = a.norm_w ? 1 : 0;
    if (g.cl) {
        if (nm) return launch_pdl_cluster(gemm_mma_kernel<NG, EPI_RESID, 1, true>, grid, block, smem, s, (int)grid.x, a, g, status);
        return launch_pdl_cluster(gemm_mma_kernel<NG, EPI_RESID, 0, true>, grid, block, smem, s, (int)grid.x, a, g, status);
    }
#define MM(ep, n) if (a.epi == ep && nm == n) return launch_pdl(gemm_mma_kernel<NG, ep, n>, grid, block, smem, s, a, g, status)
    MM(EPI_STORE, 1); MM(EPI_STORE, 0); MM(EPI_RESID, 1); MM(EPI_RESID, 0); MM(EPI_SWIGLU, 1); MM(EPI_SWIGLU, 0);
#undef MM
    return cudaErrorInvalidValue;
}

template <int R, int WR>
cudaError_t launch_rw(const GemvArgs &a, const GemvGeo &g, size_t smem, int32_t *status, cudaStream_t s) {
    return launch_pdl(gemv_kernel<R, WR>, dim3(g.S0 + g.S1, g.NR), dim3(GV_THREADS), smem, s, a, g, status);
}
template <int R, int WR, int EPI, int NORMED, bool SEG>
cudaError_t launch_lean(const GemvArgs &a, const GemvGeo &g, size_t smem, int32_t *status, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemv_kernel<R, WR, true, EPI, NORMED, SEG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(224 * 1024));
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemv_kernel<R, WR, true, EPI, NORMED, SEG>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_pdl(gemv_kernel<R, WR, true, EPI, NORMED, SEG>, dim3(g.S0 + g.S1, g.NR), dim3(GV_THREADS), smem, s, a, g, status);
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace

cudaError_t configure_gemv() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (g_sms < 1) g_sms = 148;
    // every kernel asks for the largest shared-memory carve-out, so that an SM never has to drain to
    // re-partition L1/shared memory before a CTA of the next kernel can join the running one
#define CFG(r, w) if (e == cudaSuccess) e = cudaFuncSetAttribute(gemv_kernel<r, w>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GV_SMEM_MAX); \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemv_kernel<r, w>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared)
    CFG(1, 4); CFG(2, 4); CFG(3, 4); CFG(4, 4); CFG(1, 8); CFG(2, 8); CFG(3, 8); CFG(4, 8);
#undef CFG
#define CFGM(n, ep, nm) if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_mma_kernel<n, ep, nm>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GV_SMEM_MAX); \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_mma_kernel<n, ep, nm>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared)
#define CFGM6(n) CFGM(n, EPI_STORE, 1); CFGM(n, EPI_STORE, 0); CFGM(n, EPI_RESID, 1); CFGM(n, EPI_RESID, 0); CFGM(n, EPI_SWIGLU, 1); CFGM(n, EPI_SWIGLU, 0)
    CFGM6(1); CFGM6(2);
#undef CFGM6
#undef CFGM
#define CFGC(n, nm) if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_mma_kernel<n, EPI_RESID, nm, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GV_SMEM_MAX); \
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_mma_kernel<n, EPI_RESID, nm, true>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared)
    CFGC(1, 0); CFGC(1, 1); CFGC(2, 0); CFGC(2, 1);
#undef CFGC
    // how many clusters of 2, 3, 4 CTAs the GPU runs at once with one such CTA per SM: the CTAs of a cluster share a
    // GPC, so this can be fewer than SMs / size; row ranges are sized so that every cluster is resident at once
    for (int S = 2; S <= HS_H_PARTS && e == cudaSuccess; ++S) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(S, g_sms / S); cfg.blockDim = dim3(GV_THREADS); cfg.dynamicSmemBytes = GV_SMEM_MAX;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = S; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_mma_kernel<2, EPI_RESID, 1, true>, &cfg) == cudaSuccess && n > 0) g_max_clusters[S] = n;
        else { g_max_clusters[S] = 0; cudaGetLastError(); }
        if (getenv("HS_VERBOSE")) fprintf(stderr, "libhs: clusters of %d CTAs resident at once: %d\n", S, g_max_clusters[S]);
    }
    return e;
}

// Launches the projection.  a.max_oparts > 1 allows a K split for the residual epilogue; the number
// of parts written is returned in *oparts (1 for the other epilogues).
bool gemv_uses_tc(int nrows, bool have_xb) { return (nrows > GV_MAXROWS || nrows >= g_hs_tc_min_rows) && g_hs_gemm_tc && have_xb; }

cudaError_t launch_gemv(const GemvArgs &a_in, int32_t *status, cudaStream_t s, int64_t *launches, int *oparts) {
    GemvArgs a = a_in;
    // Pulling the next projection's weights into L2 pays while they are a small part of it (measured: 4-17 MB matrices
    // gain 2 % per step); 26-105 MB matrices push each other out of the 126 MB L2 before they are used and are then
    // read from HBM twice (a 3B-class draft step: 2.21 ms with the prefetch, 1.87 ms without)
    if (a.pf_bytes > ((int64_t)20 << 20)) a.pf_bytes = 0;
    // One to three activation rows: the CUDA-core kernel.  4..16 rows: the tensor-core kernel.  More rows go in several
    // launches (the weights are streamed again for each).  g_hs_gemm_mma = false sends everything through the
    // CUDA-core kernel (passes of at most four rows over resident tiles; four rows per launch when a K range
    // needs more than one chunk).
    auto rows_launch = [&](int step) -> cudaError_t {
        for (int r = 0; r < a.nrows; r += step) {
            GemvArgs b = a;
            b.nrows = a.nrows - r < step ? a.nrows - r : step;
            b.x0 = a.x0 + (size_t)r * a.ldx0;
            if (a.x1) b.x1 = a.x1 + (size_t)r * a.ldx1;
            b.out = a.out + (size_t)r * a.ldo;
            if (a.resid) b.resid = a.resid + (size_t)r * a.ldo;
            cudaError_t e = launch_gemv(b, status, s, launches, oparts);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    };
    const bool mma = g_hs_gemm_mma && a.nrows >= 4;       // measured: up to three rows the pruned FMA instances are faster
    if (gemv_uses_tc(a.nrows, a.xb != nullptr)) return launch_gemm_tc(a, status, s, launches, oparts);   // a dense contraction: tcgen05
    if (a.nrows > GV_MAXROWS) return rows_launch(GV_MAXROWS);
    if (!mma && a.nrows > 4) {
        const int K = a.K0 > a.K1 ? a.K0 : a.K1;
        const bool splittable = a.epi == EPI_RESID && a.max_oparts > 1;
        if ((splittable ? (a.K0 + a.K1 + 3) / 4 : K) > 1280) return rows_launch(4);
    }
    if ((a.K0 & 255) || (a.K1 & 255) || a.K0 < 256 || a.O < 2 || a.nrows < 1 || a.nrows > GV_MAXROWS) return cudaErrorInvalidValue;
    GemvGeo g{};
    g.unit = a.epi == EPI_SWIGLU ? 2 : 1;
    if (a.O % g.unit) return cudaErrorInvalidValue;
    const int maxp = (a.epi == EPI_RESID && a.max_oparts > 1) ? (a.max_oparts < 4 ? a.max_oparts : 4) : 1;
    // K split: ranges of about 1024 columns, at most maxp in total, aligned to the segment boundary
    if (maxp == 1) {
        if (a.K1) return cudaErrorInvalidValue;               // two segments need at least two parts
        g.S0 = 1; g.S1 = 0;
    } else {
        for (int krt = 1024;; krt += 256) {
            g.S0 = ceil_div(a.K0, krt); g.S1 = a.K1 ? ceil_div(a.K1, krt) : 0;
            if (g.S0 + g.S1 <= maxp) break;
        }
    }
    g.kr0 = ceil_div(ceil_div(a.K0, g.S0), 256) * 256;
    g.kr1 = g.S1 ? ceil_div(ceil_div(a.K1, g.S1), 256) * 256 : 0;
    g.S0 = ceil_div(a.K0, g.kr0);
    if (g.S1) g.S1 = ceil_div(a.K1, g.kr1);
    g.krmax = g.kr0 > g.kr1 ? g.kr0 : g.kr1;
    const int S = g.S0 + g.S1;
    const int units = a.O / g.unit;
    g.NR = g_sms / S;
    // many activation rows: the consumers of a split residual stream re-add its parts for every row in every CTA,
    // which costs more than reducing the K split here, inside a cluster
    g.cl = (g_hs_cluster_reduce && mma && a.epi == EPI_RESID && S > 1 && S <= HS_H_PARTS && g_max_clusters[S] > 0) ? 1 : 0;
    if (g.cl && g.NR > g_max_clusters[S]) g.NR = g_max_clusters[S];
    if (g.NR < 1) g.NR = 1;
    if (g.NR > units) g.NR = units;
    const int nrow_max = ceil_div(units, g.NR) * g.unit;
    // tile: 4 weight rows per warp when that already gives every warp a tile, else 8
    // (wide K ranges: 4-row tiles of whole rows - requests of several KB stream best)
    const int WR = mma ? 8 : ((nrow_max <= 4 * GV_WARPS || g.krmax > 1280) ? 4 : 8);
    const int NG = a.nrows <= 8 ? 1 : 2;                       // tensor-core kernel: groups of 8 activation rows
    const int tpad = mma ? 8 : 0;                              // its tile rows are padded by 16 bytes
    // chunk of at most 1280 columns, as even as possible; narrower if the ring would not fit
    const size_t xs = mma ? (size_t)NG * 16 * (g.krmax + 8) * 2 : (size_t)a.nrows * g.krmax * 4;
    g.off_x = 1024;
    g.off_nw = (int)((g.off_x + xs + 127) / 128 * 128);
    g.off_ring = g.off_nw + (a.norm_w ? g.krmax * 4 : 0);
    const int ring_warps = ceil_div(nrow_max, WR) < GV_WARPS ? ceil_div(nrow_max, WR) : GV_WARPS;
    size_t tile = 0;
    for (int nch = mma ? ceil_div(g.krmax, 1280) : 1;; ++nch) {
        g.kc = ceil_div(ceil_div(g.krmax, nch), 256) * 256;
        tile = (size_t)WR * (g.kc + tpad) * 2;
        if (g.off_ring + tile * ring_warps <= GV_SMEM_MAX || g.kc == 256) break;
    }
    const int nchunks = ceil_div(g.krmax, g.kc);
    g.nch = nchunks; g.rq = units / g.NR; g.rrem = units % g.NR;
    g.pf_per = ((a.pf_bytes / ((int64_t)g.NR * S)) + 15) & ~15ll;
    if (!mma && a.nrows > 4 && nchunks > 1) return rows_launch(4);   // passes need every chunk of a row group resident
    const int tiles_per_warp = ceil_div(ceil_div(nrow_max, WR), GV_WARPS) * nchunks;
    int D = 1;
    const size_t budget = g.off_ring + tile * GV_WARPS > GV_SMEM_PAIR ? GV_SMEM_MAX : GV_SMEM_PAIR;   // no room for a neighbour anyway: go deep
    while (D < GV_MAXDEPTH && D < tiles_per_warp && g.off_ring + tile * GV_WARPS * (D + 1) <= budget) ++D;
    g.D = D;
    size_t smem = g.off_ring + tile * ring_warps * D;
    if (g.cl) { g.off_part = (int)((smem + 127) / 128 * 128); smem = g.off_part + (size_t)nrow_max * GV_MAXROWS * 4; }
    if (smem > GV_SMEM_MAX) return a.nrows > 1 ? rows_launch((a.nrows + 1) / 2) : cudaErrorInvalidValue;
    if (oparts) *oparts = (a.epi == EPI_RESID && !g.cl) ? S : 1;
    if (launches) ++*launches;
    if (mma) return NG == 1 ? launch_mma<1>(a, g, smem, status, s) : launch_mma<2>(a, g, smem, status, s);
    if (a.nrows <= 3) {
        // one to three rows: the pruned instances (rows, tile height, epilogue, norm fixed at compile time)
        const int nm = a.norm_w ? 1 : 0;
#define LEAN(r, w, ep, n) if (a.nrows == r && WR == w && a.epi == ep && nm == n) {                                         \
        if (ep == EPI_RESID && g.S1 > 0) return launch_lean<r, w, ep, n, ep == EPI_RESID>(a, g, smem, status, s);          \
        if (g.S1 == 0) return launch_lean<r, w, ep, n, false>(a, g, smem, status, s); }
#define LEAN6(r, w) LEAN(r, w, EPI_STORE, 1); LEAN(r, w, EPI_STORE, 0); LEAN(r, w, EPI_RESID, 1); LEAN(r, w, EPI_RESID, 0); \
                    LEAN(r, w, EPI_SWIGLU, 1); LEAN(r, w, EPI_SWIGLU, 0)
        LEAN6(1, 4); LEAN6(1, 8); LEAN6(2, 4); LEAN6(2, 8); LEAN6(3, 4); LEAN6(3, 8);
#undef LEAN6
#undef LEAN
    }
    // rows held in registers per pass: as even as possible over ceil(nrows / 4) passes
    const int npass = ceil_div(a.nrows, 4), R = ceil_div(a.nrows, npass);
#define CASE(r, w) if (R == r && WR == w) return launch_rw<r, w>(a, g, smem, status, s)
    CASE(1, 4); CASE(2, 4); CASE(3, 4); CASE(4, 4); CASE(1, 8); CASE(2, 8); CASE(3, 8); CASE(4, 8);
#undef CASE
    return cudaErrorInvalidValue;
}

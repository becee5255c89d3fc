// Recurrent mixers of the hybrid block, for T = 1 (draft step) or T = k+1 (verify) positions:
//   * Mamba-2 branch: causal conv (width 4) + SiLU on x|B|C, softplus(dt), the state recurrence
//       S <- exp(dt A) S + dt x (x) B ,  y = S C + D x ,  then the gate y * silu(z)
//   * Gated DeltaNet layer: conv + SiLU on q|k|v, L2-normalised q,k, the delta rule
//       S <- a S ; S <- S + b (v - S k) k^T ; o = S q / sqrt(dk), per-head RMSNorm and gate.
// The state of a (sequence, head, row strip) lives in registers for the whole kernel: it is read
// once with 128-bit loads, advanced T times, and written after every position (verify: one
// snapshot per position, so that rollback is an index; draft: the scratch copy).  Reductions over
// the state dimension are warp shuffles in a fixed order.
#include "hs_internal.h"
#include "hs_device.cuh"
#include "ssm_body.cuh"

namespace {
using namespace hsd;

template <int EPL, int SSM_PR, int TMAX>
__global__ void __launch_bounds__(SSM_THREADS) ssm_kernel(const SsmArgs a) {
    ssm_body<EPL, SSM_PR, TMAX>(a, blockIdx.x, blockIdx.y, blockIdx.z);
}

// ------------------------------------------------------------------------------------------------
constexpr int GDN_THREADS = 256;   // 8 warps x 8 value rows; key dim 64 = 32 lanes x 2

// TMAX: most positions this instance handles (1 for the draft step, 3 for verify at k <= 2, else the maximum).
// Everything the block needs from the in-projection - the raw conv inputs of a thread's own channel for all
// positions, the gate inputs, the decay / write-strength inputs - is requested right after the wait, before the
// first value is used: one trip to L2 for the whole kernel.
template <int TMAX>
__global__ void __launch_bounds__(GDN_THREADS) gdn_kernel(const GdnArgs a) {
    constexpr int DK = 64, RPW = 8;
    __shared__ __align__(16) float qs[TMAX][DK], ks[TMAX][DK];
    __shared__ float vs[TMAX][64], os[TMAX][64], zs[TMAX][64], al[TMAX], be[TMAX];
    const int h = blockIdx.x, lb = blockIdx.y, b = a.b0 + lb, T = TMAX == 1 ? 1 : a.T, dv = a.dv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, rowbase = lb * T;
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait
    const int nk = a.gh * DK, nv = a.gh * dv;

    const int cslot = (a.in_slot_stride || a.out_rel) ? __ldcg(a.slot + b) : 0;
    if ((unsigned)cslot >= (unsigned)a.nslot) {     // a control word out of range is never turned into an address
        if (threadIdx.x == 0) atomicCAS(a.status, 0, (int)HS_ERR_DEVICE);
        return;
    }
    const int islot = a.slot_mod ? (cslot + a.in_add) % a.slot_mod : cslot;
    const float *sin_ = a.state_in + (size_t)b * a.in_seq_stride + (a.in_slot_stride ? (size_t)islot * a.in_slot_stride : 0) + (size_t)h * dv * DK;
    float s[RPW][2];
    const bool rows_ok = warp * RPW < dv;
    // before the wait the state is only pulled towards L2 (it was written by an earlier kernel); it is loaded
    // after the wait, so this kernel may start as early as its predecessor allows.  Conv parameters are weights.
    if (rows_ok)
#pragma unroll
        for (int r = 0; r < RPW; ++r) asm volatile("prefetch.global.L2 [%0];" :: "l"(sin_ + (warp * RPW + r) * DK + 2 * lane));
    const int c = threadIdx.x;                        // this thread's channel of the head's q | k | v set
    const bool chan = c < 2 * DK + dv;
    const int gc = c < DK ? h * DK + c : c < 2 * DK ? nk + h * DK + (c - DK) : 2 * nk + h * dv + (c - 2 * DK);
    float4 tap = make_float4(0.f, 0.f, 0.f, 0.f);
    float bias = 0.f;
    if (chan) { tap = *reinterpret_cast<const float4 *>(a.conv_w + 4 * gc); bias = a.conv_b[gc]; }
    pdl_wait();
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        float2 t = rows_ok ? __ldcg(reinterpret_cast<const float2 *>(sin_ + (warp * RPW + r) * DK + 2 * lane)) : make_float2(0.f, 0.f);
        s[r][0] = t.x; s[r][1] = t.y;
    }
    float w0 = 0.f, w1 = 0.f, w2 = 0.f, raw[TMAX];
    if (chan) {
        const float *win = a.win_in + (size_t)b * 3 * a.convd + gc;
        w0 = __ldcg(win); w1 = __ldcg(win + a.convd); w2 = __ldcg(win + 2 * a.convd);
    }
#pragma unroll
    for (int i = 0; i < TMAX; ++i) raw[i] = (chan && i < T) ? __ldcg(a.zx + (size_t)(rowbase + i) * a.in_ld + gc) : 0.f;
    constexpr int ZPT = (TMAX * 64 + GDN_THREADS - 1) / GDN_THREADS;
    float zraw[ZPT];
#pragma unroll
    for (int u = 0; u < ZPT; ++u) {
        const int idx = threadIdx.x + u * GDN_THREADS, i = idx >> 6, j = idx & 63;
        zraw[u] = (i < T && j < dv) ? __ldcg(a.zx + (size_t)(rowbase + i) * a.in_ld + 2 * nk + nv + h * dv + j) : 0.f;
    }
    float araw = 0.f, braw = 0.f;
    if (threadIdx.x < T) {
        const float *row = a.zx + (size_t)(rowbase + threadIdx.x) * a.in_ld;
        araw = __ldcg(row + 2 * nk + 2 * nv + h);
        braw = __ldcg(row + 2 * nk + 2 * nv + a.gh + h);
    }
    // conv + SiLU on this head's q, k, v channels, in registers
    if (chan) {
#pragma unroll
        for (int i = 0; i < TMAX; ++i) {
            if (i < T) {
                const float r = raw[i];
                const float act = silu_f(bias + tap.x * w0 + tap.y * w1 + tap.z * w2 + tap.w * r);
                w0 = w1; w1 = w2; w2 = r;
                if (c < DK) qs[i][c] = act; else if (c < 2 * DK) ks[i][c - DK] = act; else vs[i][c - 2 * DK] = act;
                if (a.hist) a.hist[((size_t)b * a.Tm + i) * a.convd + gc] = r;
            }
        }
        if (a.win_out) {
            float *wo = a.win_out + (size_t)b * 3 * a.convd + gc;
            wo[0] = w0; wo[a.convd] = w1; wo[2 * a.convd] = w2;
        }
    }
#pragma unroll
    for (int u = 0; u < ZPT; ++u) {
        const int idx = threadIdx.x + u * GDN_THREADS, i = idx >> 6, j = idx & 63;
        if (i < T && j < dv) zs[i][j] = silu_f(zraw[u]);
    }
    if (threadIdx.x < T) { al[threadIdx.x] = sigmoid_f(araw); be[threadIdx.x] = sigmoid_f(braw); }
    __syncthreads();
    // L2-normalise q and k of every position (one warp per vector)
    for (int t = warp; t < 2 * T; t += GDN_THREADS / 32) {
        float *vec = t < T ? qs[t] : ks[t - T];
        float x0 = vec[2 * lane], x1 = vec[2 * lane + 1];
        float inv = rsqrtf(warp_sum(x0 * x0 + x1 * x1) + 1e-6f);
        vec[2 * lane] = x0 * inv; vec[2 * lane + 1] = x1 * inv;
    }
    __syncthreads();

    // rollback by replay: log the operands of every update (alpha, beta, normalised k, v) instead of storing states
    if (a.log) {
        float *lg = a.log + (size_t)b * a.Tm * a.log_w;
        for (int idx = threadIdx.x; idx < T * (DK + 64); idx += GDN_THREADS) {
            const int i = idx / (DK + 64), c = idx - i * (DK + 64);
            if (c < DK) lg[(size_t)i * a.log_w + 2 * a.gh + h * DK + c] = ks[i][c];
            else if (c - DK < dv) lg[(size_t)i * a.log_w + 2 * a.gh + nk + h * dv + (c - DK)] = vs[i][c - DK];
        }
        if (threadIdx.x < T) {
            lg[(size_t)threadIdx.x * a.log_w + h] = al[threadIdx.x];
            lg[(size_t)threadIdx.x * a.log_w + a.gh + h] = be[threadIdx.x];
        }
    }
    float *sout = a.state_out + (size_t)b * a.out_seq_stride + (size_t)h * dv * DK;
    constexpr int LPV = 32 / RPW;
    for (int i = 0; i < T; ++i) {
        const float alpha = al[i], beta = be[i];
        const float k0 = ks[i][2 * lane], k1 = ks[i][2 * lane + 1], q0 = qs[i][2 * lane], q1 = qs[i][2 * lane + 1];
        float part[RPW];
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            s[r][0] *= alpha; s[r][1] *= alpha;
            part[r] = fmaf(s[r][0], k0, s[r][1] * k1);
        }
        const float rk = xreduce<RPW>(part, lane);          // S' k for row lane / LPV
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const float rr = __shfl_sync(0xffffffffu, rk, r * LPV);
            const float u = beta * ((rows_ok ? vs[i][warp * RPW + r] : 0.f) - rr);
            s[r][0] = fmaf(u, k0, s[r][0]); s[r][1] = fmaf(u, k1, s[r][1]);
            part[r] = fmaf(s[r][0], q0, s[r][1] * q1);
        }
        const float o = xreduce<RPW>(part, lane);
        if (rows_ok && (lane & (LPV - 1)) == 0) os[i][warp * RPW + lane / LPV] = o * 0.125f;   // 1/sqrt(64)
        if (rows_ok && !a.log) {
            const int oslot = a.out_rel ? (cslot + a.out_add + i) % a.slot_mod : i;
            float *dst = sout + (size_t)oslot * a.out_slot_stride;
#pragma unroll
            for (int r = 0; r < RPW; ++r)
                *reinterpret_cast<float2 *>(dst + (warp * RPW + r) * DK + 2 * lane) = make_float2(s[r][0], s[r][1]);
        }
    }
    __syncthreads();
    // per-head RMSNorm over dv, then the output gate silu(z)
    for (int i = warp; i < T; i += GDN_THREADS / 32) {
        float ss = 0.f;
        for (int j = lane; j < dv; j += 32) ss = fmaf(os[i][j], os[i][j], ss);
        const float rstd = rsqrtf(warp_sum(ss) / (float)dv + a.eps);
        for (int j = lane; j < dv; j += 32)
            a.g[(size_t)(rowbase + i) * nv + h * dv + j] = os[i][j] * rstd * a.onorm[j] * zs[i][j];
    }
}

// ------------------------------------------------------------------------------------------------
// Rollback by replay.  The verify pass logged the operands of its k+1 state updates; once the accept kernel has
// fixed n, the first n + 1 of them are applied to the committed state in place, with the very operations (and
// operand values) the verify pass used in registers, so the result equals the snapshot it would have stored.
// One launch covers every recurrent layer: grid z = layer * sequences.
template <int EPL>
__global__ void __launch_bounds__(SSM_THREADS) replay_ssm_kernel(const ReplayArgs a) {
    constexpr int N = 32 * EPL, PR = 16, RPW = PR / (SSM_THREADS / 32);
    constexpr int VW = EPL < 4 ? EPL : 4, NVEC = EPL / VW;
    const int p0 = blockIdx.x * PR, h = blockIdx.y, rl = blockIdx.z / a.nb, lb = blockIdx.z - rl * a.nb, b = a.b0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_trigger();
    float *sp = a.state + ((size_t)rl * a.B + b) * a.state_elems + ((size_t)h * a.P + p0 + warp * RPW) * N;
    const float *lg = a.log + ((size_t)rl * a.B + b) * a.Tm * a.log_w;
    pdl_wait();
    const int n = __ldcg(a.n_acc + b);
    if ((unsigned)n >= (unsigned)a.Tm) {            // the log holds Tm entries
        if (threadIdx.x == 0) atomicCAS(a.status, 0, (int)HS_ERR_DEVICE);
        return;
    }
    float s[RPW][EPL];
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int v = 0; v < NVEC; ++v) {
            const float *src = sp + r * N + v * (32 * VW) + lane * VW;
            if (VW == 4) { float4 t = __ldcg(reinterpret_cast<const float4 *>(src)); s[r][v * 4] = t.x; s[r][v * 4 + 1] = t.y; s[r][v * 4 + 2] = t.z; s[r][v * 4 + 3] = t.w; }
            else { float2 t = __ldcg(reinterpret_cast<const float2 *>(src)); s[r][0] = t.x; s[r][1] = t.y; }
        }
#pragma unroll 1
    for (int i = 0; i <= n; ++i) {
        const float *li = lg + (size_t)i * a.log_w;
        const float dec = __ldcg(li + h);
        float Bv[EPL];
#pragma unroll
        for (int v = 0; v < NVEC; ++v)
#pragma unroll
            for (int j = 0; j < VW; ++j) Bv[v * VW + j] = __ldcg(li + a.H + a.di + v * (32 * VW) + lane * VW + j);
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const float dtx = __ldcg(li + a.H + h * a.P + p0 + warp * RPW + r);
#pragma unroll
            for (int e = 0; e < EPL; ++e) s[r][e] = fmaf(dec, s[r][e], dtx * Bv[e]);
        }
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int v = 0; v < NVEC; ++v) {
            float *p = sp + r * N + v * (32 * VW) + lane * VW;
            if (VW == 4) *reinterpret_cast<float4 *>(p) = make_float4(s[r][v * 4], s[r][v * 4 + 1], s[r][v * 4 + 2], s[r][v * 4 + 3]);
            else *reinterpret_cast<float2 *>(p) = make_float2(s[r][0], s[r][1]);
        }
}

__global__ void __launch_bounds__(GDN_THREADS) replay_gdn_kernel(const ReplayArgs a) {
    constexpr int DK = 64, RPW = 8, LPV = 32 / RPW;
    const int h = blockIdx.x, rl = blockIdx.y / a.nb, lb = blockIdx.y - rl * a.nb, b = a.b0 + lb, dv = a.dv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nk = a.gh * DK;
    pdl_trigger();
    float *sp = a.state + ((size_t)rl * a.B + b) * a.state_elems + (size_t)h * dv * DK;
    const float *lg = a.log + ((size_t)rl * a.B + b) * a.Tm * a.log_w;
    const bool rows_ok = warp * RPW < dv;
    pdl_wait();
    const int n = __ldcg(a.n_acc + b);
    if ((unsigned)n >= (unsigned)a.Tm) {            // the log holds Tm entries
        if (threadIdx.x == 0) atomicCAS(a.status, 0, (int)HS_ERR_DEVICE);
        return;
    }
    float s[RPW][2];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        float2 t = rows_ok ? __ldcg(reinterpret_cast<const float2 *>(sp + (warp * RPW + r) * DK + 2 * lane)) : make_float2(0.f, 0.f);
        s[r][0] = t.x; s[r][1] = t.y;
    }
#pragma unroll 1
    for (int i = 0; i <= n; ++i) {
        const float *li = lg + (size_t)i * a.log_w;
        const float alpha = __ldcg(li + h), beta = __ldcg(li + a.gh + h);
        const float k0 = __ldcg(li + 2 * a.gh + h * DK + 2 * lane), k1 = __ldcg(li + 2 * a.gh + h * DK + 2 * lane + 1);
        float part[RPW];
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            s[r][0] *= alpha; s[r][1] *= alpha;
            part[r] = fmaf(s[r][0], k0, s[r][1] * k1);
        }
        const float rk = xreduce<RPW>(part, lane);
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const float rr = __shfl_sync(0xffffffffu, rk, r * LPV);
            const float u = beta * ((rows_ok ? __ldcg(li + 2 * a.gh + nk + h * dv + warp * RPW + r) : 0.f) - rr);
            s[r][0] = fmaf(u, k0, s[r][0]); s[r][1] = fmaf(u, k1, s[r][1]);
        }
    }
    if (rows_ok)
#pragma unroll
        for (int r = 0; r < RPW; ++r)
            *reinterpret_cast<float2 *>(sp + (warp * RPW + r) * DK + 2 * lane) = make_float2(s[r][0], s[r][1]);
}

}  // namespace

cudaError_t launch_replay(const ReplayArgs &a, cudaStream_t s) {
    if (a.n_rl < 1) return cudaSuccess;
    if (a.arch == HS_ARCH_PARALLEL) {
        const dim3 grid(a.P / 16, a.H, a.nb * a.n_rl);
        if (a.N == 64) return launch_pdl(replay_ssm_kernel<2>, grid, dim3(SSM_THREADS), 0, s, a);
        if (a.N == 128) return launch_pdl(replay_ssm_kernel<4>, grid, dim3(SSM_THREADS), 0, s, a);
        if (a.N == 256) return launch_pdl(replay_ssm_kernel<8>, grid, dim3(SSM_THREADS), 0, s, a);
        return cudaErrorInvalidValue;
    }
    return launch_pdl(replay_gdn_kernel, dim3(a.gh, a.nb * a.n_rl), dim3(GDN_THREADS), 0, s, a);
}

// a whole head per block once blocks of 16 rows would already fill the GPU several times over
bool ssm_wide(const SsmArgs &a) { return a.P % 64 == 0 && (int64_t)(a.P / 16) * a.H * a.nb >= 148 * 32; }

cudaError_t launch_ssm(const SsmArgs &a, cudaStream_t s) {
    const bool wide = ssm_wide(a);
    const dim3 grid(a.P / (wide ? 64 : 16), a.H, a.nb);
#define LAUNCH(e_, pr_, t_) launch_pdl(ssm_kernel<e_, pr_, t_>, grid, dim3(SSM_THREADS), 0, s, a)
#define CASE(n_, e_) if (a.N == n_) return a.T == 1 ? (wide ? LAUNCH(e_, 64, 1) : LAUNCH(e_, 16, 1))               \
                                         : a.T <= 3 ? (wide ? LAUNCH(e_, 64, 3) : LAUNCH(e_, 16, 3))               \
                                                    : (wide ? LAUNCH(e_, 64, HS_MAX_T) : LAUNCH(e_, 16, HS_MAX_T))
    CASE(64, 2); CASE(128, 4); CASE(256, 8);
#undef CASE
#undef LAUNCH
    return cudaErrorInvalidValue;
}

cudaError_t launch_gdn(const GdnArgs &a, cudaStream_t s) {
    if (a.dk != 64 || a.dv > 64 || (a.dv & 7)) return cudaErrorInvalidValue;
    const dim3 grid(a.gh, a.nb), block(GDN_THREADS);
    if (a.T == 1) return launch_pdl(gdn_kernel<1>, grid, block, 0, s, a);
    if (a.T <= 3) return launch_pdl(gdn_kernel<3>, grid, block, 0, s, a);
    return launch_pdl(gdn_kernel<HS_MAX_T>, grid, block, 0, s, a);
}

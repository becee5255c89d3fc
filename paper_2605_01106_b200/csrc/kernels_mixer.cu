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

    const float *sin_ = a.state_in + (size_t)b * a.in_seq_stride +
                        (a.in_slot_stride ? (size_t)__ldcg(a.slot + b) * a.in_slot_stride : 0) + (size_t)h * dv * DK;
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
        if (rows_ok) {
            float *dst = sout + (size_t)i * a.out_slot_stride;
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

}  // namespace

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

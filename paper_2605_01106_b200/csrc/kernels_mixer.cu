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

namespace {
using namespace hsd;

constexpr int SSM_THREADS = 128; // 4 warps x PR / 4 rows

// EPL: floats of one state row held by a lane (N = 32 * EPL).  SSM_PR: state rows (of P) per block - 16
// spreads one sequence over many blocks; 64 (a whole head) is for large batches, where the conv of the
// shared B and C channels, redone by every block, would otherwise outweigh the state traffic.
template <int EPL, int SSM_PR>
__global__ void __launch_bounds__(SSM_THREADS) ssm_kernel(SsmArgs a) {
    constexpr int N = 32 * EPL;
    constexpr int VW = EPL < 4 ? EPL : 4;       // vector width of the state loads
    constexpr int NVEC = EPL / VW;
    constexpr int RPW = SSM_PR / (SSM_THREADS / 32);
    __shared__ __align__(16) float Bs[HS_MAX_T][N], Cs[HS_MAX_T][N];
    __shared__ float xs[HS_MAX_T][SSM_PR], dt_s[HS_MAX_T], a_s[HS_MAX_T];

    const int p0 = blockIdx.x * SSM_PR, h = blockIdx.y, lb = blockIdx.z, b = a.b0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, T = a.T;
    const int rowbase = lb * T;
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait

    // ---- before the wait only parameters are read; the recurrent state (written by an earlier kernel of
    //      the step or of the previous round) is merely pulled towards L2 and loaded after the wait, together
    //      with the in-projection's outputs, so that this kernel may start as early as its predecessor allows
    const float *sin_ = a.state_in + (size_t)b * a.in_seq_stride +
                        (a.in_slot_stride ? (size_t)__ldcg(a.slot + b) * a.in_slot_stride : 0) +
                        ((size_t)h * a.P + p0 + warp * RPW) * N;
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int v = 0; v < NVEC; ++v)
            asm volatile("prefetch.global.L2 [%0];" :: "l"(sin_ + r * N + v * (32 * VW) + lane * VW));
    float s[RPW][EPL];
    // ---- still before the wait: the conv parameters.
    // A thread owns the channels tid, tid + 128, ... of this block's set: its x strip, all of B and C.
    constexpr int NCH = SSM_PR + 2 * N;
    constexpr int CPT = (NCH + SSM_THREADS - 1) / SSM_THREADS;
    __shared__ float zs[HS_MAX_T][SSM_PR];
    const bool owner = (blockIdx.x == 0 && blockIdx.y == 0);   // writes the shared B|C channels' history
    float4 tap[CPT];
    float bias[CPT], w0[CPT], w1[CPT], w2[CPT];
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
        const int c = threadIdx.x + q * SSM_THREADS;
        if (c < NCH) {
            const int gc = c < SSM_PR ? h * a.P + p0 + c : a.di + (c - SSM_PR);
            tap[q] = *reinterpret_cast<const float4 *>(a.conv_w + 4 * gc);
            bias[q] = a.conv_b[gc];
        }
    }
    const float Aexp = expf(a.A_log[h]), dtb = a.dt_bias[h], Dh = a.D[h];
    pdl_wait();

    // ---- after the wait: the state rows and the conv window (L2 hits), in flight with the sweep below
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int v = 0; v < NVEC; ++v) {
            const float *src = sin_ + r * N + v * (32 * VW) + lane * VW;
            if (VW == 4) { float4 t = __ldcg(reinterpret_cast<const float4 *>(src)); s[r][v * 4] = t.x; s[r][v * 4 + 1] = t.y; s[r][v * 4 + 2] = t.z; s[r][v * 4 + 3] = t.w; }
            else { float2 t = __ldcg(reinterpret_cast<const float2 *>(src)); s[r][0] = t.x; s[r][1] = t.y; }
        }
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
        const int c = threadIdx.x + q * SSM_THREADS;
        if (c < NCH) {
            const int gc = c < SSM_PR ? h * a.P + p0 + c : a.di + (c - SSM_PR);
            const float *win = a.win_in + (size_t)b * 3 * a.convd + gc;
            w0[q] = __ldcg(win); w1[q] = __ldcg(win + a.convd); w2[q] = __ldcg(win + 2 * a.convd);
        }
    }
    // ---- raw conv inputs, gate inputs and dt of all T positions: one sweep of independent loads
    for (int idx = threadIdx.x; idx < T * NCH; idx += SSM_THREADS) {
        const int i = idx / NCH, c = idx - i * NCH;
        const int gc = c < SSM_PR ? h * a.P + p0 + c : a.di + (c - SSM_PR);
        const float raw = __ldcg(a.zx + (size_t)(rowbase + i) * a.in_ld + a.di + gc);
        if (c < SSM_PR) xs[i][c] = raw;
        else if (c < SSM_PR + N) Bs[i][c - SSM_PR] = raw;
        else Cs[i][c - SSM_PR - N] = raw;
    }
    for (int idx = threadIdx.x; idx < T * SSM_PR; idx += SSM_THREADS) {
        const int i = idx / SSM_PR, c = idx - i * SSM_PR;
        zs[i][c] = __ldcg(a.zx + (size_t)(rowbase + i) * a.in_ld + h * a.P + p0 + c);
    }
    if (threadIdx.x < T) {
        const float dt = softplus_f(__ldcg(a.zx + (size_t)(rowbase + threadIdx.x) * a.in_ld + a.di + a.convd + h) + dtb);
        dt_s[threadIdx.x] = dt;
        a_s[threadIdx.x] = expf(-dt * Aexp);
    }
    __syncthreads();
    // ---- causal conv + SiLU in place (one thread walks the positions of its channel)
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
        const int c = threadIdx.x + q * SSM_THREADS;
        if (c < NCH) {
            const int gc = c < SSM_PR ? h * a.P + p0 + c : a.di + (c - SSM_PR);
            float *col = c < SSM_PR ? &xs[0][c] : c < SSM_PR + N ? &Bs[0][c - SSM_PR] : &Cs[0][c - SSM_PR - N];
            const int stride = c < SSM_PR ? SSM_PR : N;
            const bool wr = c < SSM_PR || owner;
            float v0 = w0[q], v1 = w1[q], v2 = w2[q];
            for (int i = 0; i < T; ++i) {
                const float raw = col[i * stride];
                col[i * stride] = silu_f(bias[q] + tap[q].x * v0 + tap[q].y * v1 + tap[q].z * v2 + tap[q].w * raw);
                v0 = v1; v1 = v2; v2 = raw;
                if (wr && a.hist) a.hist[((size_t)b * a.Tm + i) * a.convd + gc] = raw;
            }
            if (wr && a.win_out) {
                float *wo = a.win_out + (size_t)b * 3 * a.convd + gc;
                wo[0] = v0; wo[a.convd] = v1; wo[2 * a.convd] = v2;
            }
        }
    }
    __syncthreads();

    // ---- recurrence over the T positions
    float *sout = a.state_out + (size_t)b * a.out_seq_stride + ((size_t)h * a.P + p0 + warp * RPW) * N;
    for (int i = 0; i < T; ++i) {
        const float dec = a_s[i], dt = dt_s[i];
        float Bv[EPL], Cv[EPL];
#pragma unroll
        for (int v = 0; v < NVEC; ++v)
#pragma unroll
            for (int j = 0; j < VW; ++j) {
                Bv[v * VW + j] = Bs[i][v * (32 * VW) + lane * VW + j];
                Cv[v * VW + j] = Cs[i][v * (32 * VW) + lane * VW + j];
            }
        float acc[RPW];
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const float dtx = dt * xs[i][warp * RPW + r];
            float t = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                s[r][e] = fmaf(dec, s[r][e], dtx * Bv[e]);
                t = fmaf(s[r][e], Cv[e], t);
            }
            acc[r] = t;
        }
        const float y = xreduce<RPW>(acc, lane);           // lanes l with l / (32/RPW) == r hold row r
        constexpr int LPV = 32 / RPW;
        if ((lane & (LPV - 1)) == 0) {
            const int r = lane / LPV, col = h * a.P + p0 + warp * RPW + r;
            const float z = zs[i][warp * RPW + r];
            a.g[(size_t)(rowbase + i) * a.di + col] = (y + Dh * xs[i][warp * RPW + r]) * silu_f(z);
        }
        // state after position i (verify: snapshot i; draft: the scratch state)
        float *dst = sout + (size_t)i * a.out_slot_stride;
#pragma unroll
        for (int r = 0; r < RPW; ++r)
#pragma unroll
            for (int v = 0; v < NVEC; ++v) {
                float *p = dst + r * N + v * (32 * VW) + lane * VW;
                if (VW == 4) *reinterpret_cast<float4 *>(p) = make_float4(s[r][v * 4], s[r][v * 4 + 1], s[r][v * 4 + 2], s[r][v * 4 + 3]);
                else *reinterpret_cast<float2 *>(p) = make_float2(s[r][0], s[r][1]);
            }
    }
}

// ------------------------------------------------------------------------------------------------
constexpr int GDN_THREADS = 256;   // 8 warps x 8 value rows; key dim 64 = 32 lanes x 2

__global__ void __launch_bounds__(GDN_THREADS) gdn_kernel(GdnArgs a) {
    constexpr int DK = 64, RPW = 8;
    __shared__ __align__(16) float qs[HS_MAX_T][DK], ks[HS_MAX_T][DK];
    __shared__ float vs[HS_MAX_T][64], os[HS_MAX_T][64], al[HS_MAX_T], be[HS_MAX_T];
    const int h = blockIdx.x, lb = blockIdx.y, b = a.b0 + lb, T = a.T, dv = a.dv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, rowbase = lb * T;
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait
    const int nk = a.gh * DK, nv = a.gh * dv;

    const float *sin_ = a.state_in + (size_t)b * a.in_seq_stride +
                        (a.in_slot_stride ? (size_t)__ldcg(a.slot + b) * a.in_slot_stride : 0) + (size_t)h * dv * DK;
    float s[RPW][2];
    const bool rows_ok = warp * RPW < dv;
    // before the wait the state is only pulled towards L2 (it was written by an earlier kernel); it is loaded
    // after the wait, so this kernel may start as early as its predecessor allows
    if (rows_ok)
#pragma unroll
        for (int r = 0; r < RPW; ++r) asm volatile("prefetch.global.L2 [%0];" :: "l"(sin_ + (warp * RPW + r) * DK + 2 * lane));
    pdl_wait();
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        float2 t = rows_ok ? __ldcg(reinterpret_cast<const float2 *>(sin_ + (warp * RPW + r) * DK + 2 * lane)) : make_float2(0.f, 0.f);
        s[r][0] = t.x; s[r][1] = t.y;
    }
    // conv + SiLU on this head's q, k, v channels
    for (int c = threadIdx.x; c < 2 * DK + dv; c += GDN_THREADS) {
        const int gc = c < DK ? h * DK + c : c < 2 * DK ? nk + h * DK + (c - DK) : 2 * nk + h * dv + (c - 2 * DK);
        const float4 tap = *reinterpret_cast<const float4 *>(a.conv_w + 4 * gc);
        const float bias = a.conv_b[gc];
        const float *win = a.win_in + (size_t)b * 3 * a.convd + gc;
        float w0 = __ldcg(win), w1 = __ldcg(win + a.convd), w2 = __ldcg(win + 2 * a.convd);
        for (int i = 0; i < T; ++i) {
            const float raw = __ldcg(a.zx + (size_t)(rowbase + i) * a.in_ld + gc);
            const float act = silu_f(bias + tap.x * w0 + tap.y * w1 + tap.z * w2 + tap.w * raw);
            w0 = w1; w1 = w2; w2 = raw;
            if (c < DK) qs[i][c] = act; else if (c < 2 * DK) ks[i][c - DK] = act; else vs[i][c - 2 * DK] = act;
            if (a.hist) a.hist[((size_t)b * a.Tm + i) * a.convd + gc] = raw;
        }
        if (a.win_out) {
            float *wo = a.win_out + (size_t)b * 3 * a.convd + gc;
            wo[0] = w0; wo[a.convd] = w1; wo[2 * a.convd] = w2;
        }
    }
    if (threadIdx.x < T) {
        const float *row = a.zx + (size_t)(rowbase + threadIdx.x) * a.in_ld;
        al[threadIdx.x] = sigmoid_f(__ldcg(row + 2 * nk + 2 * nv + h));
        be[threadIdx.x] = sigmoid_f(__ldcg(row + 2 * nk + 2 * nv + a.gh + h));
    }
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
        const float *row = a.zx + (size_t)(rowbase + i) * a.in_ld;
        for (int j = lane; j < dv; j += 32) {
            const float z = __ldcg(row + 2 * nk + nv + h * dv + j);
            a.g[(size_t)(rowbase + i) * nv + h * dv + j] = os[i][j] * rstd * a.onorm[j] * silu_f(z);
        }
    }
}

}  // namespace

cudaError_t launch_ssm(const SsmArgs &a, cudaStream_t s) {
    // a whole head per block once blocks of 16 rows would already fill the GPU several times over
    const bool wide = a.P % 64 == 0 && (int64_t)(a.P / 16) * a.H * a.nb >= 148 * 32;
    const dim3 grid(a.P / (wide ? 64 : 16), a.H, a.nb);
#define CASE(n_, e_) if (a.N == n_) return wide ? launch_pdl(ssm_kernel<e_, 64>, grid, dim3(SSM_THREADS), 0, s, a) \
                                                 : launch_pdl(ssm_kernel<e_, 16>, grid, dim3(SSM_THREADS), 0, s, a)
    CASE(64, 2); CASE(128, 4); CASE(256, 8);
#undef CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_gdn(const GdnArgs &a, cudaStream_t s) {
    if (a.dk != 64 || a.dv > 64 || (a.dv & 7)) return cudaErrorInvalidValue;
    return launch_pdl(gdn_kernel, dim3(a.gh, a.nb), dim3(GDN_THREADS), 0, s, a);
}

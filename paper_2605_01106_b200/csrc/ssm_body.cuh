// Mamba-2 mixer block body (conv + SiLU + softplus + state recurrence + gate), shared by the stand-alone
// mixer kernel and the fused mixer + attention kernel of the verify pass.
#pragma once
#include "hs_internal.h"
#include "hs_device.cuh"

namespace hsd {

constexpr int SSM_THREADS = 128; // 4 warps x PR / 4 rows

// EPL: floats of one state row held by a lane (N = 32 * EPL).  SSM_PR: state rows (of P) per block - 16
// spreads one sequence over many blocks; 64 (a whole head) is for large batches, where the conv of the
// shared B and C channels, redone by every block, would otherwise outweigh the state traffic.
// The body takes its block coordinates as arguments: (row strip, head, local sequence); it is also one of the
// two roles of the fused mixer + attention launch of the verify pass.
// TMAX: most positions this instance handles (1 for the draft step: a much shorter program, which matters
// because every launch of a step starts with a cold instruction cache).
template <int EPL, int SSM_PR, int TMAX>
__device__ __forceinline__ void ssm_body(const SsmArgs &a, const int bx, const int by, const int bz) {
    constexpr int N = 32 * EPL;
    constexpr int VW = EPL < 4 ? EPL : 4;       // vector width of the state loads
    constexpr int NVEC = EPL / VW;
    constexpr int RPW = SSM_PR / (SSM_THREADS / 32);
    __shared__ __align__(16) float Bs[TMAX][N], Cs[TMAX][N];
    __shared__ float xs[TMAX][SSM_PR], dt_s[TMAX], a_s[TMAX];

    const int p0 = bx * SSM_PR, h = by, lb = bz, b = a.b0 + lb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, T = TMAX == 1 ? 1 : a.T;
    const int rowbase = lb * T;
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait

    // ---- before the wait only parameters are read; the recurrent state (written by an earlier kernel of
    //      the step or of the previous round) is merely pulled towards L2 and loaded after the wait, together
    //      with the in-projection's outputs, so that this kernel may start as early as its predecessor allows
    const int cslot = (a.in_slot_stride || a.out_rel) ? __ldcg(a.slot + b) : 0;
    if ((unsigned)cslot >= (unsigned)a.nslot) {     // a control word out of range is never turned into an address
        if (threadIdx.x == 0) atomicCAS(a.status, 0, (int)HS_ERR_DEVICE);
        return;
    }
    const int islot = a.slot_mod ? (cslot + a.in_add) % a.slot_mod : cslot;
    const float *sin_ = a.state_in + (size_t)b * a.in_seq_stride + (a.in_slot_stride ? (size_t)islot * a.in_slot_stride : 0) +
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
    __shared__ float zs[TMAX][SSM_PR];
    const bool owner = (bx == 0 && by == 0);   // writes the shared B|C channels' history
    float4 tap[CPT];
    float bias[CPT], w0[CPT], w1[CPT], w2[CPT];
    // addresses of everything read after the wait are formed here, so that the loads go out back to back
    const float *raw_p[CPT], *win_p[CPT];
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
        const int c = threadIdx.x + q * SSM_THREADS;
        const int gc = c < SSM_PR ? h * a.P + p0 + c : a.di + (c - SSM_PR);
        raw_p[q] = a.zx + (size_t)rowbase * a.in_ld + a.di + gc;
        win_p[q] = a.win_in + (size_t)b * 3 * a.convd + gc;
        if (c < NCH) {
            tap[q] = *reinterpret_cast<const float4 *>(a.conv_w + 4 * gc);
            bias[q] = a.conv_b[gc];
        }
    }
    constexpr int ZPT = (TMAX * SSM_PR + SSM_THREADS - 1) / SSM_THREADS;
    const float *z_p[ZPT];
#pragma unroll
    for (int u = 0; u < ZPT; ++u) {
        const int idx = threadIdx.x + u * SSM_THREADS, i = idx / SSM_PR, c = idx - i * SSM_PR;
        z_p[u] = a.zx + (size_t)(rowbase + i) * a.in_ld + h * a.P + p0 + c;
    }
    const float *dt_p = a.zx + (size_t)(rowbase + threadIdx.x) * a.in_ld + a.di + a.convd + h;
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
        if (c < NCH) { w0[q] = __ldcg(win_p[q]); w1[q] = __ldcg(win_p[q] + a.convd); w2[q] = __ldcg(win_p[q] + 2 * a.convd); }
    }
    // ---- raw conv inputs of this thread's own channels for all T positions, gate inputs and dt: every load is
    //      issued before the first value is used, so the whole phase costs one trip to L2
    float raw[CPT][TMAX];
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
        const int c = threadIdx.x + q * SSM_THREADS;
#pragma unroll
        for (int i = 0; i < TMAX; ++i)
            raw[q][i] = (c < NCH && i < T) ? __ldcg(raw_p[q] + (size_t)i * a.in_ld) : 0.f;
    }
    float zraw[ZPT];
#pragma unroll
    for (int u = 0; u < ZPT; ++u)
        zraw[u] = threadIdx.x + u * SSM_THREADS < T * SSM_PR ? __ldcg(z_p[u]) : 0.f;
    const float dtraw = threadIdx.x < T ? __ldcg(dt_p) : 0.f;
    // ---- causal conv + SiLU in registers (a thread walks the positions of its channels); results to shared memory
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
        const int c = threadIdx.x + q * SSM_THREADS;
        if (c < NCH) {
            const int gc = c < SSM_PR ? h * a.P + p0 + c : a.di + (c - SSM_PR);
            float *col = c < SSM_PR ? &xs[0][c] : c < SSM_PR + N ? &Bs[0][c - SSM_PR] : &Cs[0][c - SSM_PR - N];
            const int stride = c < SSM_PR ? SSM_PR : N;
            const bool wr = c < SSM_PR || owner;
            float v0 = w0[q], v1 = w1[q], v2 = w2[q];
#pragma unroll
            for (int i = 0; i < TMAX; ++i) {
                if (i < T) {
                    const float r = raw[q][i];
                    col[i * stride] = silu_f(bias[q] + tap[q].x * v0 + tap[q].y * v1 + tap[q].z * v2 + tap[q].w * r);
                    v0 = v1; v1 = v2; v2 = r;
                    if (wr && a.hist) a.hist[((size_t)b * a.Tm + i) * a.convd + gc] = r;
                }
            }
            if (wr && a.win_out) {
                float *wo = a.win_out + (size_t)b * 3 * a.convd + gc;
                wo[0] = v0; wo[a.convd] = v1; wo[2 * a.convd] = v2;
            }
        }
    }
#pragma unroll
    for (int u = 0; u < ZPT; ++u) {
        const int idx = threadIdx.x + u * SSM_THREADS, i = idx / SSM_PR, c = idx - i * SSM_PR;
        if (idx < T * SSM_PR) zs[i][c] = zraw[u];
    }
    if (threadIdx.x < T) {
        const float dt = softplus_f(dtraw + dtb);
        dt_s[threadIdx.x] = dt;
        a_s[threadIdx.x] = expf(-dt * Aexp);
    }
    __syncthreads();

    // ---- rollback by replay: instead of a state per position, the verify pass leaves what each update needs - the
    //      head's decay, this strip's dt * x and (one block per sequence) the shared B - exactly the operands of the
    //      recurrence below, so that replaying them reproduces its states bit for bit
    if (a.log) {
        float *lg = a.log + (size_t)b * a.Tm * a.log_w;
        for (int idx = threadIdx.x; idx < T * SSM_PR; idx += SSM_THREADS) {
            const int i = idx / SSM_PR, c = idx - i * SSM_PR;
            lg[(size_t)i * a.log_w + a.H + h * a.P + p0 + c] = dt_s[i] * xs[i][c];
        }
        if (bx == 0 && threadIdx.x < T) lg[(size_t)threadIdx.x * a.log_w + h] = a_s[threadIdx.x];
        if (owner)
            for (int idx = threadIdx.x; idx < T * N; idx += SSM_THREADS) {
                const int i = idx / N, n = idx - i * N;
                lg[(size_t)i * a.log_w + a.H + a.di + n] = Bs[i][n];
            }
    }

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
        // state after position i (verify: snapshot i; draft: the scratch state; rollback by replay: nothing)
        if (a.log) continue;
        const int oslot = a.out_rel ? (cslot + a.out_add + i) % a.slot_mod : i;
        float *dst = sout + (size_t)oslot * a.out_slot_stride;
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


}  // namespace hsd

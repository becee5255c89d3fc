// Skinny projection kernels: out[r][o] = sum_j W[o][j] * x[r][j] for a handful of activation rows r
// (batch * (k+1)), bf16 weights streamed once from HBM, fp32 activations and accumulation.
//
// The work is HBM-bound (every weight byte is used R <= 9 times), so it runs on the CUDA cores:
// a warp owns WR consecutive weight rows and walks the K dimension with 128-bit streaming loads;
// the R activation rows (after an optional fused RMSNorm) sit in shared memory and are re-used by
// all WR rows; the WR*R partial sums of a lane are combined with a transposing shuffle reduction
// (WR*R - 1 shuffles instead of 5 per value, fixed order -> bit-reproducible).
// Epilogues: plain store, residual add, SwiGLU over interleaved gate/up rows.
#include "hs_internal.h"
#include "hs_device.cuh"

namespace {
using namespace hsd;

__device__ __forceinline__ float dot8(const uint4 &w, const float4 &a, const float4 &b, float acc) {
    acc = fmaf(bf_lo(w.x), a.x, acc); acc = fmaf(bf_hi(w.x), a.y, acc);
    acc = fmaf(bf_lo(w.y), a.z, acc); acc = fmaf(bf_hi(w.y), a.w, acc);
    acc = fmaf(bf_lo(w.z), b.x, acc); acc = fmaf(bf_hi(w.z), b.y, acc);
    acc = fmaf(bf_lo(w.w), b.z, acc); acc = fmaf(bf_hi(w.w), b.w, acc);
    return acc;
}

template <int R, int WR>
__global__ void __launch_bounds__(256) gemv_kernel(GemvArgs a) {
    constexpr int NV = pow2_ge(R * WR);
    extern __shared__ __align__(16) float smem[];
    const int Kt = a.K0 + a.K1;
    const int nw = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float *x_s = smem;                    // [R][Kt]
    float *res_s = smem + R * Kt;         // [nw][32]
    float *rstd_s = res_s + nw * 32;      // [R]

    for (int rb = 0; rb < a.nrows; rb += R) {
        const int nr = min(R, a.nrows - rb);
        // ---- stage the activation rows (zero rows beyond nr)
        const int q4 = Kt >> 2, q0 = a.K0 >> 2;
        for (int idx = threadIdx.x; idx < R * q4; idx += blockDim.x) {
            int r = idx / q4, c = idx - r * q4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < nr) {
                if (c < q0) v = *reinterpret_cast<const float4 *>(a.x0 + (size_t)(rb + r) * a.ldx0 + 4 * c);
                else v = *reinterpret_cast<const float4 *>(a.x1 + (size_t)(rb + r) * a.ldx1 + 4 * (c - q0));
            }
            *reinterpret_cast<float4 *>(x_s + r * Kt + 4 * c) = v;
        }
        __syncthreads();
        if (a.norm_w) {
            // fused RMSNorm of segment 0: x <- x * rsqrt(mean(x^2) + eps) * w
            for (int r = warp; r < R; r += nw) {
                float ss = 0.f;
                for (int j = lane; j < a.K0; j += 32) { float t = x_s[r * Kt + j]; ss = fmaf(t, t, ss); }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                if (lane == 0) rstd_s[r] = rsqrtf(ss / (float)a.K0 + a.eps);
            }
            __syncthreads();
            for (int idx = threadIdx.x; idx < R * a.K0; idx += blockDim.x) {
                int r = idx / a.K0, j = idx - r * a.K0;
                x_s[r * Kt + j] *= rstd_s[r] * a.norm_w[j];
            }
            __syncthreads();
        }
        // ---- stream the weights
        for (int og = (blockIdx.x * nw + warp) * WR; og < a.O; og += gridDim.x * nw * WR) {
            float acc[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) acc[i] = 0.f;
#pragma unroll
            for (int seg = 0; seg < 2; ++seg) {
                const __nv_bfloat16 *W = seg ? a.W1 : a.W0;
                const int K = seg ? a.K1 : a.K0, ld = seg ? a.ldw1 : a.ldw0, koff = seg ? a.K0 : 0;
                if (K == 0) continue;
                const __nv_bfloat16 *wrow[WR];
#pragma unroll
                for (int w = 0; w < WR; ++w) wrow[w] = W + (size_t)min(og + w, a.O - 1) * ld;
#pragma unroll 2
                for (int kc = lane * 8; kc < K; kc += 256) {
                    uint4 wv[WR];
#pragma unroll
                    for (int w = 0; w < WR; ++w) wv[w] = ldg_stream(wrow[w] + kc);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        const float4 xa = *reinterpret_cast<const float4 *>(x_s + r * Kt + koff + kc);
                        const float4 xb = *reinterpret_cast<const float4 *>(x_s + r * Kt + koff + kc + 4);
#pragma unroll
                        for (int w = 0; w < WR; ++w) acc[r * WR + w] = dot8(wv[w], xa, xb, acc[r * WR + w]);
                    }
                }
            }
            const float tot = xreduce<NV>(acc, lane);
            constexpr int LPV = 32 / NV;                     // lanes that hold each value
            if ((lane & (LPV - 1)) == 0) res_s[warp * 32 + lane / LPV] = tot;
            __syncwarp();
            // ---- epilogue: value index = r * WR + w
            if (a.epi == EPI_SWIGLU) {
                if (lane < nr * (WR / 2)) {
                    int r = lane / (WR / 2), p = lane - r * (WR / 2);
                    int o = og + 2 * p;
                    if (o + 1 < a.O) {
                        float gt = res_s[warp * 32 + r * WR + 2 * p], up = res_s[warp * 32 + r * WR + 2 * p + 1];
                        a.out[(size_t)(rb + r) * a.ldo + (o >> 1)] = silu_f(gt) * up;
                    }
                }
            } else {
                if (lane < nr * WR) {
                    int r = lane / WR, w = lane - r * WR;
                    int o = og + w;
                    if (o < a.O) {
                        float v = res_s[warp * 32 + r * WR + w];
                        size_t oi = (size_t)(rb + r) * a.ldo + o;
                        if (a.epi == EPI_RESID) v += a.resid[oi];
                        a.out[oi] = v;
                    }
                }
            }
            __syncwarp();
        }
        __syncthreads();
    }
}

constexpr size_t GEMV_SMEM_MAX = 201 * 1024;

template <int R, int WR>
cudaError_t launch_t(const GemvArgs &a, int nw, int grid, size_t smem, cudaStream_t s) {
    gemv_kernel<R, WR><<<grid, nw * 32, smem, s>>>(a);
    return cudaGetLastError();
}

template <int R, int WR>
cudaError_t configure_t() {
    return cudaFuncSetAttribute(gemv_kernel<R, WR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMV_SMEM_MAX);
}

}  // namespace

// Opt every instantiation into large dynamic shared memory once, outside any stream capture.
cudaError_t configure_gemv() {
    cudaError_t e = cudaSuccess;
#define CFG(r, w) if (e == cudaSuccess) e = configure_t<r, w>()
    CFG(1, 2); CFG(2, 2); CFG(3, 2); CFG(4, 2); CFG(5, 2); CFG(9, 2);
    CFG(1, 4); CFG(2, 4); CFG(3, 4); CFG(4, 4); CFG(5, 4);
#undef CFG
    return e;
}

cudaError_t launch_gemv(const GemvArgs &a, cudaStream_t s, int64_t *launches) {
    const int Kt = a.K0 + a.K1;
    if ((a.K0 & 255) || (a.K1 & 255) || a.O < 2 || a.nrows < 1) return cudaErrorInvalidValue;
    // rows per pass: must fit shared memory; fewest passes, then smallest R
    static const int cand[6] = {1, 2, 3, 4, 5, 9};
    int R = 1, best_pass = 1 << 30;
    for (int i = 0; i < 6; ++i) {
        size_t bytes = (size_t)cand[i] * Kt * 4 + 8 * 32 * 4 + 64;
        if (bytes > 200 * 1024) continue;
        int pass = (a.nrows + cand[i] - 1) / cand[i];
        if (pass < best_pass) { best_pass = pass; R = cand[i]; }
    }
    int WR = (R * 4 <= 32 && a.O >= 4096) ? 4 : 2;
    int nw = (a.O / WR >= 148 * 8) ? 8 : 4;
    int grid = (a.O + nw * WR - 1) / (nw * WR);
    if (grid > 148 * 8) grid = 148 * 8;
    size_t smem = (size_t)R * Kt * 4 + nw * 32 * 4 + 64;
    if (launches) ++*launches;
#define CASE(r, w) if (R == r && WR == w) return launch_t<r, w>(a, nw, grid, smem, s)
    CASE(1, 2); CASE(2, 2); CASE(3, 2); CASE(4, 2); CASE(5, 2); CASE(9, 2);
    CASE(1, 4); CASE(2, 4); CASE(3, 4); CASE(4, 4); CASE(5, 4);
#undef CASE
    return cudaErrorInvalidValue;
}

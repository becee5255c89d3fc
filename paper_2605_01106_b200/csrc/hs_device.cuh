// Device helpers shared by the kernels of libhs.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace hsd {

// 128-bit streaming load: read-only path, no L1 allocation (weights and KV rows are used once)
__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// the two bf16 halves of a 32-bit word as fp32 (exact)
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + expf(-x)); }
__device__ __forceinline__ float sigmoid_f(float x) { return 1.0f / (1.0f + expf(-x)); }
__device__ __forceinline__ float softplus_f(float x) { return x > 20.0f ? x : log1pf(expf(x)); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Transposing warp reduction.  Every lane holds NV partial sums (NV a power of two <= 32);
// afterwards the lanes l with l / (32/NV) == i hold the warp-wide total of value i.
// NV - 1 + log2(32/NV) shuffles, fixed summation order.
template <int NV>
__device__ __forceinline__ float xreduce(float (&v)[NV], int lane) {
    int off = 16;
#pragma unroll
    for (int cnt = NV; cnt > 1; cnt >>= 1) {
        const int half = cnt >> 1;
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            float keep = up ? v[i + half] : v[i];
            float send = up ? v[i] : v[i + half];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
        off >>= 1;
    }
    float r = v[0];
#pragma unroll
    for (int o = 32 / NV / 2; o >= 1; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
    return r;
}

__host__ __device__ constexpr int pow2_ge(int x) { return x <= 1 ? 1 : x <= 2 ? 2 : x <= 4 ? 4 : x <= 8 ? 8 : x <= 16 ? 16 : 32; }

}  // namespace hsd

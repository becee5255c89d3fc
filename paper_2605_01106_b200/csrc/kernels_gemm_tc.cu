// Projection for many activation rows (batch * (k+1) > 16): a dense contraction, run on the fifth-generation
// tensor cores.  out[r][o] = sum_j W[o][j] x[r][j] is computed as D = A B^T with
//   A = a 128-row tile of the weight matrix (bf16, K-major), streamed by TMA tensor copies into 128-byte
//       swizzled shared-memory stages,
//   B = the activation rows, packed once per projection by a small kernel into bf16 head and bf16 remainder
//       planes (x = head + remainder to 2^-17, with the RMSNorm weight and 1/rms folded in); a CTA takes BNH
//       rows of each plane (all rows when there are at most 128) as the N = 2 * BNH columns of its tile,
//   D = 128 x N fp32 accumulators in tensor memory; the epilogue reads them back with tcgen05.ld, adds the head
//       and remainder columns and applies the store / residual / SwiGLU epilogue.
// One elected thread issues the TMA copies, one issues tcgen05.mma (K = 16 per instruction, four per 64-column
// stage) and releases stages with tcgen05.commit; all eight warps run the epilogue (thread = weight row, two
// warps per lane quarter, each half of the columns).  Every wait is bounded.
// Every CTA fetches its own tiles (no copy is shared between CTAs).
// The weights are the large operand, so the grid is filled by splitting K, not N: the CTAs of a thread-block
// cluster (up to 8) take consecutive K ranges of the same tile, leave their fp32 partial tiles in shared
// memory and add them up, in rank order, through distributed shared memory - every weight byte is fetched
// once and the result does not depend on timing.
#include "hs_internal.h"
#include "hs_device.cuh"
#include <cuda.h>
#include <cstdio>
#include <cstdlib>

namespace {
using namespace hsd;

constexpr int TC_BM = 128;          // weight rows per CTA
constexpr int TC_BK = 64;           // K columns per stage: one 128-byte swizzle atom of bf16
constexpr int TC_THREADS = 256;    // two warps per tensor-memory lane quarter: each takes half of the columns in the epilogue
constexpr int TC_MAXSTAGES = 8;

// ---- tensor maps (driver entry point fetched once; the library does not link libcuda) ----------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// 2-D bf16 tensor [rows][cols] with row stride ld (elements), box = TC_BK columns x box_rows rows, 128-byte swizzle
cudaError_t make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    if (!g_encode) return cudaErrorNotSupported;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)TC_BK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// ---- pack: fp32 activation rows -> bf16 head plane | bf16 remainder plane, [2][rpad][Kt], norm folded in -----
struct PackArgs {
    const float *x0; int ldx0, K0, xparts; int64_t xpstride; const float *norm_w; float eps;
    const float *x1; int ldx1, K1;
    __nv_bfloat16 *xb; int nrows, rpad;
};

__global__ void __launch_bounds__(256) pack_kernel(const PackArgs a) {
    const int r = blockIdx.x, Kt = a.K0 + a.K1;
    __shared__ float red[8];
    __nv_bfloat16 *hi = a.xb + (size_t)r * Kt, *lo = a.xb + ((size_t)a.rpad + r) * Kt;
    pdl_trigger();
    pdl_wait();
    if (r >= a.nrows) {                        // padding rows are zero in both planes
        for (int c = threadIdx.x * 8; c < Kt; c += blockDim.x * 8) {
            *reinterpret_cast<uint4 *>(hi + c) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4 *>(lo + c) = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    float rstd = 1.f;
    if (a.norm_w) {
        float ss = 0.f;
        for (int c = threadIdx.x * 4; c < a.K0; c += blockDim.x * 4) {
            float4 v = __ldcg(reinterpret_cast<const float4 *>(a.x0 + (size_t)r * a.ldx0 + c));
            for (int q = 1; q < a.xparts; ++q) {
                const float4 u = __ldcg(reinterpret_cast<const float4 *>(a.x0 + (size_t)q * a.xpstride + (size_t)r * a.ldx0 + c));
                v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
            }
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += red[w];
        rstd = rsqrtf(t / (float)a.K0 + a.eps);
    }
    for (int c = threadIdx.x * 4; c < Kt; c += blockDim.x * 4) {
        float4 v;
        if (c < a.K0) {
            v = __ldcg(reinterpret_cast<const float4 *>(a.x0 + (size_t)r * a.ldx0 + c));
            for (int q = 1; q < a.xparts; ++q) {
                const float4 u = __ldcg(reinterpret_cast<const float4 *>(a.x0 + (size_t)q * a.xpstride + (size_t)r * a.ldx0 + c));
                v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
            }
            if (a.norm_w) {
                const float4 nw = *reinterpret_cast<const float4 *>(a.norm_w + c);
                v.x *= nw.x * rstd; v.y *= nw.y * rstd; v.z *= nw.z * rstd; v.w *= nw.w * rstd;
            }
        } else {
            v = __ldcg(reinterpret_cast<const float4 *>(a.x1 + (size_t)r * a.ldx1 + (c - a.K0)));
        }
        const float x[4] = {v.x, v.y, v.z, v.w};
        uint32_t hw[2], lw[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const __nv_bfloat16 h0 = __float2bfloat16_rn(x[2 * e]), h1 = __float2bfloat16_rn(x[2 * e + 1]);
            const __nv_bfloat16 l0 = __float2bfloat16_rn(x[2 * e] - __bfloat162float(h0)), l1 = __float2bfloat16_rn(x[2 * e + 1] - __bfloat162float(h1));
            hw[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
            lw[e] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
        }
        *reinterpret_cast<uint2 *>(hi + c) = make_uint2(hw[0], hw[1]);
        *reinterpret_cast<uint2 *>(lo + c) = make_uint2(lw[0], lw[1]);
    }
}

// ---- the contraction ---------------------------------------------------------------------------------------
struct TcArgs {
    int O, nk0, nk1;            // output rows; 64-column K blocks of segment 0 / 1
    int nrows, rpad, bnh;       // activation rows, rows per plane of the packed operand, rows per plane per CTA
    int ns;                     // shared-memory stages (at most TC_MAXSTAGES)
    int rb;                     // K split: activation rows of a tile each rank finishes (a power of two >= 4, rb * S >= bnh)
    float *out; int ldo;
    const float *resid; int rparts; int64_t rpstride;
    int32_t *status;
    // The packed operand may come without the 1/rms factor of its RMSNorm (a projection epilogue wrote it, see
    // pk_out): then ss_in[p * rpad + r], p < ss_parts, are partial sums of squares of activation row r and the
    // factor rsqrt(sum * inv_k + eps) is applied to the finished sums of that row.
    const float *ss_in; int ss_parts; float inv_k, eps;
    // Packed output for the projection that consumes this one's result: bf16 head | remainder planes
    // [2][rpad][pk_ld] of (result * pk_nw[output row]), and (residual epilogue) the partial sums of squares
    // ss_out[weight-row tile][rpad] of the results.  nullptr: not wanted.
    __nv_bfloat16 *pk_out; int pk_ld; const float *pk_nw; float *ss_out;
    const void *pf_ptr; long long pf_bytes;     // weights of the next projection, pulled into L2 before the wait
    int off_rx, off_misc;       // shared-memory carve-up behind the stages (bytes from the aligned base)
};

__device__ __forceinline__ void tma_load_2d(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// the same for a weight tile: streamed once per step, so marked evict-first in L2
__device__ __forceinline__ void tma_load_2d_stream(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                 :: "r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(pol) : "memory");
}
// shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    const uint32_t lo = ((smem_addr >> 4) & 0x3fffu) | (1u << 16);
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return ((uint64_t)hi << 32) | lo;
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                 :: "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr));
}
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &h, __nv_bfloat16 &l) {
    h = __float2bfloat16_rn(x);
    l = __float2bfloat16_rn(x - __bfloat162float(h));
}

// Residual of eight consecutive activation rows r0..r0+7 of weight row `row` (parts added in order); the loads
// are issued early, so that their trip to L2 hides behind the wait that precedes the epilogue proper.
__device__ __forceinline__ void tc_load_resid(const TcArgs &a, float (&res)[8], int r0, int nvalid, int row) {
#pragma unroll
    for (int j = 0; j < 8; ++j) res[j] = 0.f;
    if (row >= a.O) return;
    const size_t oi = (size_t)r0 * a.ldo + row;
    for (int p = 0; p < a.rparts; ++p) {
        const float *rp = a.resid + (size_t)p * a.rpstride + oi;
#pragma unroll
        for (int j = 0; j < 8; ++j) if (j < nvalid) res[j] += __ldcg(rp + (size_t)j * a.ldo);
    }
}

// Epilogue for eight consecutive activation rows r0..r0+7 (indices inside the launch) of weight row `row`
// (v[j] = the finished sum of row r0 + j, 1/rms already applied); nvalid of them exist.  Every lane of the warp
// calls it (the SwiGLU pairing and the sums of squares shuffle).  res: the residual (tc_load_resid); nw: weight
// folded into the packed output.  Returns (residual epilogue with statistics) the warp's sum of squares of row
// r0 + lane / 4.
template <int EPI>
__device__ __forceinline__ float tc_finish8(const TcArgs &a, float (&v)[8], const float (&res)[8], int r0, int nvalid, int row, float nw, int lane) {
    if (EPI == EPI_SWIGLU) {
        // weight rows come in (gate, up) pairs held by neighbouring lanes.  The even lane finishes the even
        // columns of the pair, the odd lane the odd ones, so both lanes work and each evaluates one SiLU per two
        // columns: lanes swap what the other needs (even sends its gate of column j + 1, odd its up of column j).
        const bool odd = row & 1;
        const bool st = (row | 1) < a.O;
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const float got = __shfl_xor_sync(0xffffffffu, odd ? v[j] : v[j + 1], 1);
            const float gate = odd ? got : v[j], up = odd ? v[j + 1] : got;
            const int jj = j + (odd ? 1 : 0);
            if (st && jj < nvalid) {
                const float r = silu_f(gate) * up;
                if (a.pk_out) {
                    __nv_bfloat16 h, l;
                    split_bf16(r, h, l);
                    __nv_bfloat16 *p = a.pk_out + (size_t)(r0 + jj) * a.pk_ld + (row >> 1);
                    p[0] = h; p[(size_t)a.rpad * a.pk_ld] = l;
                } else {
                    a.out[(size_t)(r0 + jj) * a.ldo + (row >> 1)] = r;
                }
            }
        }
        return 0.f;
    } else {
        const bool st = row < a.O;
        if (EPI == EPI_RESID)
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] += res[j];
        float *p = a.out + (size_t)r0 * a.ldo + row;
#pragma unroll
        for (int j = 0; j < 8; ++j) if (st && j < nvalid) p[(size_t)j * a.ldo] = v[j];
        if (EPI == EPI_RESID && a.pk_out) {
            __nv_bfloat16 *ph = a.pk_out + (size_t)r0 * a.pk_ld + row;
            const size_t plane = (size_t)a.rpad * a.pk_ld;
            float ssq[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool live = st && j < nvalid;
                if (live) {
                    __nv_bfloat16 h, l;
                    split_bf16(v[j] * nw, h, l);
                    ph[(size_t)j * a.pk_ld] = h; ph[(size_t)j * a.pk_ld + plane] = l;
                }
                ssq[j] = live ? v[j] * v[j] : 0.f;
            }
            return xreduce<8>(ssq, lane);           // lanes 4 j .. 4 j + 3 hold the total of row r0 + j
        }
        return 0.f;
    }
}

// BN: N of the MMA = 2 * bnh (head columns, then remainder columns).  EPI: the epilogue, fixed at compile time.
template <int BN, int EPI>
__global__ void __launch_bounds__(TC_THREADS, 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mA0, const __grid_constant__ CUtensorMap mA1,
               const __grid_constant__ CUtensorMap mB, const TcArgs a) {
    constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2, B_BYTES = BN * TC_BK * 2, STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TCOLS = BN < 32 ? 32 : BN;
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
    constexpr int BNH = BN / 2;
    extern __shared__ unsigned char smraw[];
    __shared__ __align__(8) uint64_t full_bar[TC_MAXSTAGES], empty_bar[TC_MAXSTAGES], done_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int failed_s;
    const uint32_t sbase = (smem_u32(smraw) + 1023u) & ~1023u;            // swizzled tiles need 1024-byte alignment
    unsigned char *stages = smraw + (sbase - smem_u32(smraw));
    float *rx = reinterpret_cast<float *>(stages + a.off_rx);             // [S][128][rb]: partial tiles sent by the cluster's ranks
    float *rstd_s = reinterpret_cast<float *>(stages + a.off_misc);       // [BNH]
    float *nw_s = rstd_s + 128;                                           // [128]
    float *ssred = nw_s + 128;                                            // [4][BNH]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // grid = (K splits = cluster size, weight-row tiles, activation-row tiles)
    const int S = (int)gridDim.x, q = (int)blockIdx.x;
    const int m0 = blockIdx.y * TC_BM, n0h = blockIdx.z * BNH;
    const int nk = a.nk0 + a.nk1, NS = a.ns;
    const int kb0 = (int)((long long)q * nk / S), kb1 = (int)((long long)(q + 1) * nk / S), nkl = kb1 - kb0;
    pdl_trigger();
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&done_bar, 1);
        mbar_fence_init();
        failed_s = 0;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_base_s)), "r"(TCOLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // parameters (nothing a kernel writes): the weights folded into the packed output
    if (tid >= 128) {
        const int i = tid - 128;
        nw_s[i] = (a.pk_nw && m0 + i < a.O) ? a.pk_nw[m0 + i] : 1.f;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;
    // first phase of the cluster barrier: "this CTA runs" - a rank's shared memory may be written once every rank has
    // arrived here; nobody waits for it before the exchange at the end
    if (S > 1) cluster_arrive();

    if (warp == 0 && lane == 0) {
        // ---- TMA producer.  Weight tiles depend on nothing: the first stages are requested before the wait.
        auto load_a = [&](int i) {                      // i: k block relative to kb0
            const int s = i % NS, kb = kb0 + i;
            mbar_expect_tx(&full_bar[s], STAGE);
            if (kb < a.nk0) tma_load_2d_stream(stages + (size_t)s * STAGE, &mA0, kb * TC_BK, m0, &full_bar[s]);
            else tma_load_2d_stream(stages + (size_t)s * STAGE, &mA1, (kb - a.nk0) * TC_BK, m0, &full_bar[s]);
        };
        auto load_b = [&](int i) {
            const int s = i % NS, kb = kb0 + i;
            unsigned char *bs = stages + (size_t)s * STAGE + A_BYTES;
            tma_load_2d(bs, &mB, kb * TC_BK, n0h, &full_bar[s]);
            tma_load_2d(bs + (size_t)BNH * TC_BK * 2, &mB, kb * TC_BK, a.rpad + n0h, &full_bar[s]);
        };
        const int pre = nkl < NS ? nkl : NS;
        for (int i = 0; i < pre; ++i) load_a(i);
        pdl_wait();
        for (int i = 0; i < pre; ++i) load_b(i);
        for (int i = NS; i < nkl; ++i) {
            if (!mbar_wait(&empty_bar[i % NS], (uint32_t)(i / NS - 1) & 1u)) { failed_s = 1; break; }
            load_a(i);
            load_b(i);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        for (int i = 0; i < nkl; ++i) {
            const int s = i % NS;
            if (!mbar_wait(&full_bar[s], (uint32_t)(i / NS) & 1u)) { failed_s = 1; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = sbase + (uint32_t)s * STAGE;
            const uint64_t ad = umma_desc(sa), bd = umma_desc(sa + A_BYTES);
#pragma unroll
            for (int k = 0; k < TC_BK / 16; ++k)       // 32 bytes further along K per instruction (descriptor units of 16 bytes)
                umma_bf16(tmem_d, ad + 2 * k, bd + 2 * k, IDESC, (i > 0 || k > 0) ? 1u : 0u);
            umma_commit(&empty_bar[s]);                 // the stage is free once these MMAs have read it
        }
        umma_commit(&done_bar);                         // accumulators complete
    } else if (warp >= 2) {
        // ---- the other warps: pull the next projection's weights into L2, then the 1/rms factors of this tile's rows
        if (a.pf_bytes > 0) {
            const long long ncta = (long long)gridDim.x * gridDim.y * gridDim.z;
            const long long cta = ((long long)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
            const long long per = ((a.pf_bytes + ncta - 1) / ncta + 15) & ~15ll;
            const long long lo = cta * per, hi = min(lo + per, a.pf_bytes & ~15ll);
#pragma unroll 1
            for (long long o = lo + (long long)(tid - 64) * 4096; o < hi; o += (TC_THREADS - 64) * 4096)
                prefetch_l2(reinterpret_cast<const char *>(a.pf_ptr) + o, (uint32_t)min(4096ll, hi - o));
        }
        pdl_wait();
#pragma unroll 1
        for (int i = tid - 64; i < BNH; i += TC_THREADS - 64) {
            float r = 1.f;
            if (a.ss_in) {
                float t = 0.f;
                for (int p = 0; p < a.ss_parts; ++p) t += __ldcg(a.ss_in + (size_t)p * a.rpad + n0h + i);
                r = rsqrtf(t * a.inv_k + a.eps);
            }
            rstd_s[i] = r;
        }
    }
    if (warp < 2 && !(warp == 0 && lane == 0)) pdl_wait();          // the epilogue reads the residual stream
    __syncwarp();
    __syncthreads();                                    // rstd_s complete
    // ---- epilogue: thread = accumulator lane = weight row; warps w and w + 4 share a lane quarter and split
    //      the columns (activation rows)
    const int lrow = (warp & 3) * 32 + lane, half = warp >> 2;
    const int row = m0 + lrow;
    const float nw = nw_s[lrow];
    const int nact = a.nrows - n0h;                     // activation rows of this tile that exist
    const bool stats = EPI == EPI_RESID && a.pk_out != nullptr && a.ss_out != nullptr;
    // K split: rank p finishes the activation rows [p * rb, (p + 1) * rb) of the tile (rb a power of two >= 4; ranks
    // whose range lies beyond the tile finish nothing)
    const int rb = a.rb, lg_rb = 31 - __clz(rb);
    int c_lo = 0, c_n = BNH;                            // the tile's activation rows this CTA finishes
    if (S > 1) { c_lo = min(q * rb, BNH); c_n = min(rb, BNH - c_lo); }
    // first group of eight rows this thread finishes: its residual is requested now, the trip to L2 hides behind the
    // wait for the accumulators (and the exchange)
    const int first = S == 1 ? half * (BNH / 2) : c_lo + half * 8;
    float res[8];
    if (EPI == EPI_RESID) tc_load_resid(a, res, n0h + first, nact - first, row);
    const bool ok = mbar_wait(&done_bar, 0) && !failed_s;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t taddr = tmem_d + ((uint32_t)((warp & 3) * 32) << 16);
    if (!ok && tid == 0) atomicCAS(a.status, 0, (int)HS_ERR_TIMEOUT);
    if (S == 1) {
        if (ok) {
            for (int c0 = half * (BNH / 2); c0 < (half + 1) * (BNH / 2); c0 += 8) {
                uint32_t h[8], l[8];
                tmem_ld8(taddr + (uint32_t)c0, h);
                tmem_ld8(taddr + (uint32_t)(BNH + c0), l);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                float v[8], rnext[8];
                if (EPI == EPI_RESID && c0 + 8 < (half + 1) * (BNH / 2)) tc_load_resid(a, rnext, n0h + c0 + 8, nact - (c0 + 8), row);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (__uint_as_float(h[j]) + __uint_as_float(l[j])) * rstd_s[c0 + j];
                const float sq = tc_finish8<EPI>(a, v, res, n0h + c0, nact - c0, row, nw, lane);
                if (stats && (lane & 3) == 0) ssred[(warp & 3) * BNH + c0 + (lane >> 2)] = sq;
                if (EPI == EPI_RESID)
#pragma unroll
                    for (int j = 0; j < 8; ++j) res[j] = rnext[j];
            }
        }
    } else {
        // Every rank sends the matching columns of its partial tile straight into rank p's shared memory
        // ([sender][weight row][rb]: 16-byte remote stores), ONE cluster barrier, then each rank adds the S partials of
        // its rows in rank order - the result does not depend on timing.
        cluster_wait();                                 // every rank runs: its receive area may be written
        const uint32_t rx_mine = smem_u32(rx) + (uint32_t)(((q * TC_BM + lrow) * rb) * 4);
        for (int c0 = half * (BNH / 2); c0 < (half + 1) * (BNH / 2); c0 += 8) {
            uint32_t h[8], l[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) h[j] = l[j] = 0u;
            if (ok && nkl > 0) {
                tmem_ld8(taddr + (uint32_t)c0, h);
                tmem_ld8(taddr + (uint32_t)(BNH + c0), l);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            }
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(h[j]) + __uint_as_float(l[j]);
            if (rb >= 8) {
                const uint32_t dst = dsmem_addr(rx_mine + (uint32_t)((c0 & (rb - 1)) * 4), (uint32_t)(c0 >> lg_rb));
                dsmem_st_v4(dst, v[0], v[1], v[2], v[3]);
                dsmem_st_v4(dst + 16, v[4], v[5], v[6], v[7]);
            } else {                                    // rb == 4: the eight columns belong to two ranks
                const uint32_t p = (uint32_t)(c0 >> 2);
                dsmem_st_v4(dsmem_addr(rx_mine, p), v[0], v[1], v[2], v[3]);
                dsmem_st_v4(dsmem_addr(rx_mine, p + 1), v[4], v[5], v[6], v[7]);
            }
        }
        cluster_arrive(); cluster_wait();
        // eight rows at a time, alternating between the two halves of the CTA
        for (int cl0 = half * 8; cl0 < c_n; cl0 += 16) {
            const int nr = min(8, c_n - cl0);
            float v[8], rnext[8];
            if (EPI == EPI_RESID && cl0 + 16 < c_n) tc_load_resid(a, rnext, n0h + c_lo + cl0 + 16, nact - (c_lo + cl0 + 16), row);
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = 0.f;
            for (int p = 0; p < S; ++p) {
                const float4 *pr = reinterpret_cast<const float4 *>(rx + ((size_t)(p * TC_BM + lrow) * rb + cl0));
                const float4 x = pr[0];
                v[0] += x.x; v[1] += x.y; v[2] += x.z; v[3] += x.w;
                if (nr > 4) { const float4 y = pr[1]; v[4] += y.x; v[5] += y.y; v[6] += y.z; v[7] += y.w; }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] *= rstd_s[min(c_lo + cl0 + j, BNH - 1)];
            const int nvalid = min(nr, nact - (c_lo + cl0));
            const float sq = tc_finish8<EPI>(a, v, res, n0h + c_lo + cl0, nvalid, row, nw, lane);
            if (stats && (lane & 3) == 0 && (lane >> 2) < nr) ssred[(warp & 3) * BNH + c_lo + cl0 + (lane >> 2)] = sq;
            if (EPI == EPI_RESID)
#pragma unroll
                for (int j = 0; j < 8; ++j) res[j] = rnext[j];
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (stats && ok) {
        // sums of squares of the finished rows over this tile's 128 weight rows: the four lane quarters in order
        for (int i = tid; i < c_n; i += TC_THREADS) {
            const int c = c_lo + i;
            if (c < nact) a.ss_out[(size_t)blockIdx.y * a.rpad + n0h + c] = (ssred[c] + ssred[BNH + c]) + (ssred[2 * BNH + c] + ssred[3 * BNH + c]);
        }
    }
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"(TCOLS) : "memory");
}

constexpr size_t tc_stage_bytes(int bn) { return (size_t)TC_BM * TC_BK * 2 + (size_t)bn * TC_BK * 2; }
constexpr size_t TC_SMEM_MAX = 200 * 1024;
constexpr size_t TC_SMEM_PAIR = 110 * 1024;   // up to this two CTAs fit on an SM
constexpr size_t TC_MISC_BYTES = (128 + 128 + 4 * 128) * 4;
int g_tc_clusters[2][9];     // clusters of S CTAs that run at once with one CTA per SM ([0]; [1]: the same query at the smaller footprint)

template <int BN, int EPI>
cudaError_t launch_tc(const CUtensorMap &mA0, const CUtensorMap &mA1, const CUtensorMap &mB, const TcArgs &t, dim3 grid, size_t smem, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_MAX);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_pdl_cluster(gemm_tc_kernel<BN, EPI>, grid, dim3(TC_THREADS), smem, s, (int)grid.x, mA0, mA1, mB, t);
}
template <int BN>
cudaError_t launch_tc_epi(int epi, const CUtensorMap &mA0, const CUtensorMap &mA1, const CUtensorMap &mB, const TcArgs &t, dim3 grid, size_t smem, cudaStream_t s) {
    if (epi == EPI_STORE) return launch_tc<BN, EPI_STORE>(mA0, mA1, mB, t, grid, smem, s);
    if (epi == EPI_RESID) return launch_tc<BN, EPI_RESID>(mA0, mA1, mB, t, grid, smem, s);
    return launch_tc<BN, EPI_SWIGLU>(mA0, mA1, mB, t, grid, smem, s);
}

}  // namespace

bool g_hs_gemm_tc = true;
bool g_hs_tensor_maps = false;

// K or V cache of one layer as a 2-D bf16 tensor [rows][hd]: boxes of 64 columns x 128 rows, 128-byte swizzle
cudaError_t hs_make_kv_tensor_map(CUtensorMap *map, const void *base, uint64_t rows, int hd) {
    if (hd % 64) return cudaErrorInvalidValue;
    return make_map(map, base, rows, (uint64_t)hd, (uint64_t)hd, 128);
}
int g_hs_tc_min_rows = 17;

cudaError_t configure_gemm_tc() {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    g_hs_tensor_maps = true;
    e = cudaFuncSetAttribute(pack_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_tc_kernel<32, EPI_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_MAX);
    if (e != cudaSuccess) return e;
    for (int pair = 0; pair < 2; ++pair)
        for (int S = 1; S <= 8; ++S) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(S, 148 / S); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = pair ? TC_SMEM_PAIR : TC_SMEM_MAX;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = S; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_kernel<32, EPI_STORE>, &cfg) == cudaSuccess && n > 0) g_tc_clusters[pair][S] = n;
            else { g_tc_clusters[pair][S] = S == 1 ? 148 : 0; cudaGetLastError(); }
            if (getenv("HS_VERBOSE")) fprintf(stderr, "libhs: tcgen05 projection, clusters of %d CTAs (%d per SM) resident at once: %d\n", S, pair + 1, g_tc_clusters[pair][S]);
        }
    return cudaSuccess;
}

// Rows per plane per CTA (a power of two, 16..128) and rows per plane of the packed operand for nrows activation rows.
static int tc_bnh(int nrows) { int b = 16; while (b < 128 && b < nrows) b <<= 1; return b; }
int gemm_tc_rows(int nrows) { const int b = tc_bnh(nrows); return (nrows + b - 1) / b * b; }

cudaError_t launch_gemm_tc(const GemvArgs &a, int32_t *status, cudaStream_t s, int64_t *launches, int *oparts) {
    if ((!a.xb && !a.pk_in) || (a.K0 & 63) || (a.K1 & 63) || a.nrows < 1) return cudaErrorInvalidValue;
    const int Kt = a.K0 + a.K1;
    const int mtiles = (a.O + TC_BM - 1) / TC_BM, nk = Kt / TC_BK;
    // Rows per plane per CTA.  The packed operand is laid out for the largest tile (rpad rows per plane); a small
    // weight matrix is cheap to read again from L2, so its activation rows are cut into more, smaller tiles, which
    // shortens every CTA's epilogue and spares the K split (measured on 1024-wide layers: 64 rows 4 %, 128 rows 6 %,
    // 192 rows 4 % per pass; large matrices and more than 256 rows lose)
    const int rpad = gemm_tc_rows(a.nrows);
    int bnh = tc_bnh(a.nrows);
    if ((int64_t)a.O * Kt * 2 <= ((int64_t)20 << 20)) {
        const int cap = a.nrows <= 64 ? 32 : a.nrows <= 256 ? 64 : 128;
        if (bnh > cap) bnh = cap;
    }
    const int ntiles = (a.nrows + bnh - 1) / bnh;
    // K split (cluster size, 1..8): the weights are the large operand, so the grid is filled by splitting K, as long as
    // all CTAs still run at once, at most one per SM, and every CTA keeps at least two K blocks.  Rank p of a cluster
    // finishes rb activation rows of the tile (a power of two, at least four).
    const size_t stage = tc_stage_bytes(2 * bnh);
    const int tiles = mtiles * ntiles;
    // (the CTAs of a cluster share a GPC, so fewer clusters of S CTAs than SMs / S may run at once: g_tc_clusters)
    int S = 1, rb = 4;
    size_t rx_bytes = 0, budget = TC_SMEM_MAX;
    for (int cand = 1; cand <= 8; ++cand) {
        if (cand > 1 && nk / cand < 2) break;
        int crb = 4;
        while (crb * cand < bnh) crb <<= 1;
        const size_t crx = cand > 1 ? (size_t)cand * crb * TC_BM * 4 : 0;
        // Stages as deep as shared memory allows: a refill costs a trip to L2 on the critical path (measured: deep
        // stages with one CTA per SM beat two co-resident CTAs with two or three stages each).  Few activation rows
        // make the stages small: then two CTAs fit on an SM with four or more stages each, more CTAs than SMs still
        // run at once and the CTAs of the next projection can stream their weights while this one finishes.
        // More tiles than SMs would otherwise run in two rounds, the second nearly empty: there three stages are enough
        // for a pair (measured: 4-6 % per verify pass on the batched workloads; with two stages it loses again).
        const bool pair = TC_SMEM_PAIR >= 4 * stage + crx + TC_MISC_BYTES + 1024 ||
                          (tiles * cand > 148 && TC_SMEM_PAIR >= 3 * stage + crx + TC_MISC_BYTES + 1024);
        // with two CTAs per SM twice as many clusters run at once (the occupancy query is made for one per SM)
        if (cand > 1 && tiles > g_tc_clusters[0][cand] * (pair ? 2 : 1)) continue;
        if (cand > 1 && tiles * cand > (pair ? 2 * 148 : 148)) continue;
        S = cand; rb = crb; rx_bytes = crx; budget = pair ? TC_SMEM_PAIR : TC_SMEM_MAX;
    }
    const int nkl = (nk + S - 1) / S;
    int ns = (int)((budget - rx_bytes - TC_MISC_BYTES - 1024) / stage);
    if (ns > TC_MAXSTAGES) ns = TC_MAXSTAGES;
    if (ns > nkl) ns = nkl;
    if (ns < 1) return cudaErrorInvalidValue;
    size_t smem = (size_t)ns * stage + rx_bytes + TC_MISC_BYTES + 1024;
    // tensor memory is not oversubscribed: a CTA's share of the SM's shared memory is at least its share of the
    // 512 tensor-memory columns, so an allocation never has to wait for a CTA of another cluster (which could
    // itself be waiting, at its cluster barrier, for a peer queued behind this one)
    const size_t tcols = 2 * bnh < 32 ? 32 : 2 * bnh, share = (size_t)228 * 1024 * tcols / 512 + 1024;
    if (smem < share) smem = share;
    if (smem > TC_SMEM_MAX) return cudaErrorInvalidValue;
    const __nv_bfloat16 *xb = a.pk_in;
    if (!xb) {
        if ((int64_t)rpad > a.xb_rows) return cudaErrorInvalidValue;
        PackArgs p{a.x0, a.ldx0, a.K0, a.xparts, a.xpstride, a.norm_w, a.eps, a.x1, a.ldx1, a.K1, a.xb, a.nrows, rpad};
        cudaError_t e = launch_pdl(pack_kernel, dim3(rpad), dim3(256), 0, s, p);
        if (e != cudaSuccess) return e;
        if (launches) ++*launches;
        xb = a.xb;
    }
    CUtensorMap mA0, mA1, mB;
    cudaError_t e = make_map(&mA0, a.W0, a.O, a.K0, a.ldw0, TC_BM);
    if (e == cudaSuccess) e = a.K1 ? make_map(&mA1, a.W1, a.O, a.K1, a.ldw1, TC_BM) : make_map(&mA1, a.W0, a.O, a.K0, a.ldw0, TC_BM);
    if (e == cudaSuccess) e = make_map(&mB, xb, (uint64_t)2 * rpad, Kt, Kt, bnh);
    if (e != cudaSuccess) return e;
    TcArgs t{};
    t.O = a.O; t.nk0 = a.K0 / TC_BK; t.nk1 = a.K1 / TC_BK; t.nrows = a.nrows; t.rpad = rpad; t.bnh = bnh; t.ns = ns; t.rb = rb;
    t.out = a.out; t.ldo = a.ldo; t.resid = a.resid; t.rparts = a.rparts; t.rpstride = a.rpstride; t.status = status;
    if (a.pk_in && a.ss_in) { t.ss_in = a.ss_in; t.ss_parts = a.ss_parts; t.inv_k = 1.f / (float)a.K0; t.eps = a.eps; }
    if (a.pk_out && a.epi != EPI_STORE) {
        t.pk_out = a.pk_out; t.pk_ld = a.pk_ld; t.pk_nw = a.pk_nw;
        t.ss_out = a.epi == EPI_RESID ? a.ss_out : nullptr;
    }
    t.pf_ptr = a.pf_ptr; t.pf_bytes = a.pf_ptr ? (long long)a.pf_bytes : 0;
    t.off_rx = (int)((size_t)ns * stage); t.off_misc = (int)((size_t)ns * stage + rx_bytes);
    if (oparts) *oparts = 1;
    if (launches) ++*launches;
    const dim3 grid(S, mtiles, ntiles);
    switch (2 * bnh) {
        case 32: return launch_tc_epi<32>(a.epi, mA0, mA1, mB, t, grid, smem, s);
        case 64: return launch_tc_epi<64>(a.epi, mA0, mA1, mB, t, grid, smem, s);
        case 128: return launch_tc_epi<128>(a.epi, mA0, mA1, mB, t, grid, smem, s);
        default: return launch_tc_epi<256>(a.epi, mA0, mA1, mB, t, grid, smem, s);
    }
}

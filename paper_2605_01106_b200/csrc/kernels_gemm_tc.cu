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
#include <cooperative_groups.h>

namespace {
using namespace hsd;
namespace cg = cooperative_groups;

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
    float *out; int ldo;
    const float *resid; int rparts; int64_t rpstride;
    int epi;
    int32_t *status;
};

__device__ __forceinline__ void tma_load_2d(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
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

// Epilogue for eight consecutive activation rows r0..r0+7 of weight row `row` (v[j] = the finished sum of
// row r0 + j); nvalid of them exist.  Every lane of the warp calls it (the SwiGLU pairing shuffles).
template <int EPI>
__device__ __forceinline__ void tc_finish8(const TcArgs &a, float (&v)[8], int r0, int nvalid, int row) {
    if (EPI == EPI_SWIGLU) {
        // weight rows come in (gate, up) pairs held by neighbouring lanes.  The even lane finishes the even
        // columns of the pair, the odd lane the odd ones, so both lanes work and each evaluates one SiLU per two
        // columns: lanes swap what the other needs (even sends its gate of column j + 1, odd its up of column j).
        const bool odd = row & 1;
        const bool st = (row | 1) < a.O;
        float *p = a.out + (size_t)r0 * a.ldo + (row >> 1);
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const float got = __shfl_xor_sync(0xffffffffu, odd ? v[j] : v[j + 1], 1);
            const float gate = odd ? got : v[j], up = odd ? v[j + 1] : got;
            const int jj = j + (odd ? 1 : 0);
            if (st && jj < nvalid) p[(size_t)jj * a.ldo] = gate / (1.f + __expf(-gate)) * up;
        }
    } else {
        const bool st = row < a.O;
        const size_t oi = (size_t)r0 * a.ldo + row;
        if (EPI == EPI_RESID) {
            float res[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) res[j] = 0.f;
            for (int p = 0; p < a.rparts; ++p) {
                const float *rp = a.resid + (size_t)p * a.rpstride + oi;
#pragma unroll
                for (int j = 0; j < 8; ++j) if (st && j < nvalid) res[j] += __ldcg(rp + (size_t)j * a.ldo);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] += res[j];
        }
        float *p = a.out + oi;
#pragma unroll
        for (int j = 0; j < 8; ++j) if (st && j < nvalid) p[(size_t)j * a.ldo] = v[j];
    }
}

template <int BN>               // N of the MMA = 2 * bnh (head columns, then remainder columns)
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mA0, const __grid_constant__ CUtensorMap mA1,
               const __grid_constant__ CUtensorMap mB, const TcArgs a) {
    constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2, B_BYTES = BN * TC_BK * 2, STAGE = A_BYTES + B_BYTES;
    constexpr uint32_t TCOLS = BN < 32 ? 32 : BN;
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
    extern __shared__ unsigned char smraw[];
    __shared__ __align__(8) uint64_t full_bar[TC_MAXSTAGES], empty_bar[TC_MAXSTAGES], done_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int failed_s;
    const uint32_t sbase = (smem_u32(smraw) + 1023u) & ~1023u;            // swizzled tiles need 1024-byte alignment
    unsigned char *stages = smraw + (sbase - smem_u32(smraw));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // grid = (K splits = cluster size, weight-row tiles, activation-row tiles)
    const int S = (int)gridDim.x, q = (int)blockIdx.x;
    const int m0 = blockIdx.y * TC_BM, n0h = blockIdx.z * a.bnh;
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
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;

    if (warp == 0 && lane == 0) {
        // ---- TMA producer.  Weight tiles depend on nothing: the first stages are requested before the wait.
        auto load_a = [&](int i) {                      // i: k block relative to kb0
            const int s = i % NS, kb = kb0 + i;
            mbar_expect_tx(&full_bar[s], STAGE);
            if (kb < a.nk0) tma_load_2d(stages + (size_t)s * STAGE, &mA0, kb * TC_BK, m0, &full_bar[s]);
            else tma_load_2d(stages + (size_t)s * STAGE, &mA1, (kb - a.nk0) * TC_BK, m0, &full_bar[s]);
        };
        auto load_b = [&](int i) {
            const int s = i % NS, kb = kb0 + i;
            unsigned char *bs = stages + (size_t)s * STAGE + A_BYTES;
            tma_load_2d(bs, &mB, kb * TC_BK, n0h, &full_bar[s]);
            tma_load_2d(bs + (size_t)a.bnh * TC_BK * 2, &mB, kb * TC_BK, a.rpad + n0h, &full_bar[s]);
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
    }
    if (!(warp == 0 && lane == 0)) pdl_wait();          // the epilogue reads the residual stream
    __syncwarp();
    // ---- epilogue: thread = accumulator lane = weight row; warps w and w + 4 share a lane quarter and split
    //      the columns (activation rows)
    const bool ok = mbar_wait(&done_bar, 0) && !failed_s;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int lrow = (warp & 3) * 32 + lane, half = warp >> 2;
    const int row = m0 + lrow;
    const uint32_t taddr = tmem_d + ((uint32_t)((warp & 3) * 32) << 16);
    const int nact = a.nrows - n0h;                     // activation rows of this tile that exist
    auto finish8 = [&](float (&v)[8], int r0) {
        const int nvalid = nact - r0;
        if (a.epi == EPI_SWIGLU) tc_finish8<EPI_SWIGLU>(a, v, n0h + r0, nvalid, row);
        else if (a.epi == EPI_RESID) tc_finish8<EPI_RESID>(a, v, n0h + r0, nvalid, row);
        else tc_finish8<EPI_STORE>(a, v, n0h + r0, nvalid, row);
    };
    if (!ok && tid == 0) atomicCAS(a.status, 0, (int)HS_ERR_TIMEOUT);
    if (S == 1) {
        if (ok) {
            for (int c0 = half * (a.bnh / 2); c0 < (half + 1) * (a.bnh / 2); c0 += 8) {
                uint32_t h[8], l[8];
                tmem_ld8(taddr + (uint32_t)c0, h);
                tmem_ld8(taddr + (uint32_t)(a.bnh + c0), l);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(h[j]) + __uint_as_float(l[j]);
                finish8(v, c0);
            }
        }
    } else {
        // partial tile of this K range into shared memory (the stages are drained: every copy was consumed and
        // every MMA has completed), [activation row][weight row] so that both sides of the exchange are coalesced
        cg::cluster_group cluster = cg::this_cluster();
        float *red = reinterpret_cast<float *>(stages);
        for (int c0 = half * (a.bnh / 2); c0 < (half + 1) * (a.bnh / 2); c0 += 8) {
            uint32_t h[8], l[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) h[j] = l[j] = 0u;
            if (ok && nkl > 0) {
                tmem_ld8(taddr + (uint32_t)c0, h);
                tmem_ld8(taddr + (uint32_t)(a.bnh + c0), l);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) red[(c0 + j) * TC_BM + lrow] = __uint_as_float(h[j]) + __uint_as_float(l[j]);
        }
        cluster.sync();
        // rank q finishes activation rows [q * rb, (q + 1) * rb) of the tile, eight at a time (alternating between
        // the two halves of the CTA): partials added in rank order
        const int rb = a.bnh / S;
        for (int r0 = q * rb + half * 8; r0 < (q + 1) * rb; r0 += 16) {
            const int nr = min(8, (q + 1) * rb - r0);
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = 0.f;
            for (int p = 0; p < S; ++p) {
                const float *pr = cluster.map_shared_rank(red, p) + r0 * TC_BM + lrow;
#pragma unroll
                for (int j = 0; j < 8; ++j) if (j < nr) v[j] += pr[j * TC_BM];
            }
            // rows beyond nr belong to the next rank: nvalid is cut to nr inside
            float w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = v[j];
            const int nvalid = min(nr, nact - r0);
            if (a.epi == EPI_SWIGLU) tc_finish8<EPI_SWIGLU>(a, w, n0h + r0, nvalid, row);
            else if (a.epi == EPI_RESID) tc_finish8<EPI_RESID>(a, w, n0h + r0, nvalid, row);
            else tc_finish8<EPI_STORE>(a, w, n0h + r0, nvalid, row);
        }
        cluster.sync();                                  // peers may still be reading this CTA's partial
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_d), "r"(TCOLS) : "memory");
}

constexpr size_t tc_stage_bytes(int bn) { return (size_t)TC_BM * TC_BK * 2 + (size_t)bn * TC_BK * 2; }
constexpr size_t TC_SMEM_MAX = 200 * 1024;

template <int BN>
cudaError_t launch_tc(const CUtensorMap &mA0, const CUtensorMap &mA1, const CUtensorMap &mB, const TcArgs &t, dim3 grid, size_t smem, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM_MAX);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_pdl_cluster(gemm_tc_kernel<BN>, grid, dim3(TC_THREADS), smem, s, (int)grid.x, mA0, mA1, mB, t);
}

}  // namespace

bool g_hs_gemm_tc = true;

cudaError_t configure_gemm_tc() {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return cudaSuccess;
}

// Rows of scratch (per plane) a projection of nrows activation rows needs in the packed operand buffer.
int gemm_tc_rows(int nrows) { return (nrows + 127) / 128 * 128; }

cudaError_t launch_gemm_tc(const GemvArgs &a, int32_t *status, cudaStream_t s, int64_t *launches, int *oparts) {
    if (!a.xb || (a.K0 & 63) || (a.K1 & 63) || a.nrows < 1) return cudaErrorInvalidValue;
    const int Kt = a.K0 + a.K1;
    const int mtiles = (a.O + TC_BM - 1) / TC_BM, nk = Kt / TC_BK;
    // rows per plane per CTA: all of them up to 128 (power of two, at least 16)
    int bnh = 16;
    while (bnh < 128 && bnh < a.nrows) bnh <<= 1;
    const int ntiles = (a.nrows + bnh - 1) / bnh, rpad = ntiles * bnh;
    // K split (cluster size): as many CTAs as fit on the GPU at once, every CTA with at least two K blocks
    const size_t stage = tc_stage_bytes(2 * bnh);
    int S = 1;
    while (S < 8 && mtiles * ntiles * S * 2 <= 148 && nk / (S * 2) >= 2) S <<= 1;
    const int nkl = (nk + S - 1) / S;
    int ns = (int)((TC_SMEM_MAX - 1024) / stage);
    if (ns > TC_MAXSTAGES) ns = TC_MAXSTAGES;
    if (ns > nkl) ns = nkl;
    size_t smem = (size_t)ns * stage;
    if (S > 1 && smem < (size_t)bnh * TC_BM * 4) smem = (size_t)bnh * TC_BM * 4;    // room for the partial tile
    smem += 1024;
    // tensor memory is not oversubscribed: a CTA's share of the SM's shared memory is at least its share of the
    // 512 tensor-memory columns, so an allocation never has to wait for a CTA of another cluster (which could
    // itself be waiting, at its cluster barrier, for a peer queued behind this one)
    const size_t tcols = 2 * bnh < 32 ? 32 : 2 * bnh, share = (size_t)228 * 1024 * tcols / 512 + 1024;
    if (smem < share) smem = share;
    if (smem > TC_SMEM_MAX || (int64_t)rpad > a.xb_rows) return cudaErrorInvalidValue;
    PackArgs p{a.x0, a.ldx0, a.K0, a.xparts, a.xpstride, a.norm_w, a.eps, a.x1, a.ldx1, a.K1, a.xb, a.nrows, rpad};
    cudaError_t e = launch_pdl(pack_kernel, dim3(rpad), dim3(256), 0, s, p);
    if (e != cudaSuccess) return e;
    CUtensorMap mA0, mA1, mB;
    e = make_map(&mA0, a.W0, a.O, a.K0, a.ldw0, TC_BM);
    if (e == cudaSuccess) e = a.K1 ? make_map(&mA1, a.W1, a.O, a.K1, a.ldw1, TC_BM) : make_map(&mA1, a.W0, a.O, a.K0, a.ldw0, TC_BM);
    if (e == cudaSuccess) e = make_map(&mB, a.xb, (uint64_t)2 * rpad, Kt, Kt, bnh);
    if (e != cudaSuccess) return e;
    TcArgs t{a.O, a.K0 / TC_BK, a.K1 / TC_BK, a.nrows, rpad, bnh, ns, a.out, a.ldo, a.resid, a.rparts, a.rpstride, a.epi, status};
    if (oparts) *oparts = 1;
    if (launches) *launches += 2;
    const dim3 grid(S, mtiles, ntiles);
    switch (2 * bnh) {
        case 32: return launch_tc<32>(mA0, mA1, mB, t, grid, smem, s);
        case 64: return launch_tc<64>(mA0, mA1, mB, t, grid, smem, s);
        case 128: return launch_tc<128>(mA0, mA1, mB, t, grid, smem, s);
        default: return launch_tc<256>(mA0, mA1, mB, t, grid, smem, s);
    }
}

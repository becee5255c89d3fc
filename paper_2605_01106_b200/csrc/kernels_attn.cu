// Verify-mode attention: the T = k+1 new positions of a sequence attend over its KV cache plus the
// new rows themselves (causal among the new ones), grouped-query heads, split over the cache length.
//
// grid = (max splits, kv heads, sequences); one CTA = one chunk of CK cached keys for the G*T query
// rows that share its KV head (G = q heads per KV head).
//  * Before the programmatic-dependent-launch wait the CTA reads kv_len (written at least two
//    kernels earlier), starts two bulk asynchronous copies - its K chunk and its V chunk, each one
//    contiguous piece of the cache - and fetches the RoPE rows of the new positions.
//  * After the wait it rotates and scales the queries into shared memory; the CTA of the last chunk
//    also rotates the T new K rows, rounds K and V to bf16 exactly as they are cached, appends them to
//    the cache and keeps them in shared memory behind the cached keys, so nothing written by this
//    launch is read back from global memory by another block.
//  * Scores: lane = key, each warp takes a subset of the query rows; the dense key rows are read in a
//    per-lane rotated chunk order so that the 128-bit reads do not collide on a bank.  One softmax per
//    chunk (the whole chunk is resident), then P V with thread = output dimension.
//  * Several chunks: every CTA publishes an un-normalised partial (m, l, acc); the CTA that arrives
//    last (ticket counter, no spinning) merges them in chunk order, so the result is reproducible.
#include "hs_internal.h"
#include "hs_device.cuh"
#include <cooperative_groups.h>

namespace {
using namespace hsd;
namespace cg = cooperative_groups;

constexpr int AT_THREADS = 128;
constexpr int AT_WARPS = 4;
constexpr int AT_CL = 8;               // CTAs (chunks) per thread-block cluster

template <int HD>
struct AttnSmem {
    // offsets in bytes for a chunk capacity of ck cached keys (+ up to 16 new ones)
    static __host__ __device__ int keys(int ck) { return ck + 16; }
    static __host__ __device__ size_t k_off() { return 128; }
    static __host__ __device__ size_t v_off(int ck) { return k_off() + (size_t)keys(ck) * HD * 2; }
    static __host__ __device__ size_t q_off(int ck) { return v_off(ck) + (size_t)keys(ck) * HD * 2; }
    static __host__ __device__ size_t p_off(int ck) { return q_off(ck) + (size_t)HS_MAX_GT * HD * 4; }
    static __host__ __device__ size_t ml_off(int ck) { return p_off(ck) + (size_t)HS_MAX_GT * keys(ck) * 4; }
    static __host__ __device__ size_t rope_off(int ck) { return ml_off(ck) + (size_t)HS_MAX_GT * 2 * 4; }
    static __host__ __device__ size_t total(int ck) { return rope_off(ck) + (size_t)HS_MAX_T * (HD / 2) * 8; }
};

template <int HD, int GTB>      // GTB: compile-time bound of G*T (16, 32 or 48)
__global__ void __launch_bounds__(AT_THREADS) attn_kernel(const AttnArgs a) {
    using L = AttnSmem<HD>;
    constexpr int NC = HD / 8;             // 16-byte chunks per key row
    extern __shared__ __align__(128) unsigned char smraw[];
    const int CK = a.chunk;
    uint64_t *bar = reinterpret_cast<uint64_t *>(smraw);
    __nv_bfloat16 *K_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L::k_off());      // [CK + 16][HD]
    __nv_bfloat16 *V_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L::v_off(CK));
    float *q_s = reinterpret_cast<float *>(smraw + L::q_off(CK));                    // [GT][HD] rotated, pre-scaled
    float *p_s = reinterpret_cast<float *>(smraw + L::p_off(CK));                    // [GT][CK + 16]
    float *ml_s = reinterpret_cast<float *>(smraw + L::ml_off(CK));                  // [GT][2]
    float2 *rope_s = reinterpret_cast<float2 *>(smraw + L::rope_off(CK));            // [T][HD/2]
    __shared__ int ticket_s;

    const int split = blockIdx.x, kh = blockIdx.y, lb = blockIdx.z, b = a.b0 + lb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = a.qh / a.kvh, T = a.T, GT = G * T, PST = L::keys(CK);
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait

    // ---- before the wait: kv_len, the cached chunk, the RoPE rows
    const int len = __ldcg(a.kv_len + b);
    const int nsplit = max(1, (len + CK - 1) / CK);
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank(), cl = split / AT_CL;
    if (cl * AT_CL >= nsplit) return;             // the whole cluster is beyond the cache: nobody reaches a barrier
    // a CTA beyond the last chunk of a live cluster has no keys: it contributes (m, l) = (-inf, 0) and still
    // takes its share of the cluster's reduction
    const bool last = split == nsplit - 1;
    const int c0 = split * CK, ncache = max(0, min(len, c0 + CK) - c0);
    const bool overflow = len + T > a.cap;       // never write past the cache; the host reports the status word
    __nv_bfloat16 *Kb = a.Kc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    __nv_bfloat16 *Vb = a.Vc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    if (tid == 0) { mbar_init(bar, 1); mbar_fence_init(); }
    __syncthreads();
    if (tid == 0 && ncache > 0 && !overflow) {
        const uint32_t bytes = (uint32_t)ncache * HD * 2;
        mbar_expect_tx(bar, 2 * bytes);
        bulk_g2s(K_s, Kb + (size_t)c0 * HD, bytes, bar);
        bulk_g2s(V_s, Vb + (size_t)c0 * HD, bytes, bar);
    }
    if (!overflow)
        for (int idx = tid; idx < T * (HD / 2); idx += AT_THREADS) {
            const int i = idx / (HD / 2), e = idx - i * (HD / 2);
            rope_s[idx] = a.rope[(size_t)(len + i) * (HD / 2) + e];
        }
    pdl_wait();
    if (overflow) {
        if (tid == 0 && split == 0 && kh == 0) atomicCAS(a.status, 0, (int)HS_ERR_CAPACITY);
        return;
    }
    __syncthreads();                        // rope_s complete

    // ---- queries: RoPE at position len + i, pre-multiplied by 1/sqrt(hd)
    const int rowbase = lb * T;
    const float scale = rsqrtf((float)HD);
    for (int base = 0; base < GT * (HD / 2); base += AT_THREADS * 6) {
        // six elements per thread and sweep: all twelve loads are issued before the first is used
        float x0[6], x1[6];
#pragma unroll
        for (int u = 0; u < 6; ++u) {
            const int idx = base + u * AT_THREADS + tid;
            x0[u] = x1[u] = 0.f;
            if (idx < GT * (HD / 2)) {
                const int qi = idx / (HD / 2), e = idx - qi * (HD / 2);
                const int gq = qi / T, i = qi - gq * T;
                const float *src = a.zx + (size_t)(rowbase + i) * a.in_ld + a.q_off + (kh * G + gq) * HD;
                x0[u] = __ldcg(src + e); x1[u] = __ldcg(src + e + HD / 2);
            }
        }
#pragma unroll
        for (int u = 0; u < 6; ++u) {
            const int idx = base + u * AT_THREADS + tid;
            if (idx < GT * (HD / 2)) {
                const int qi = idx / (HD / 2), e = idx - qi * (HD / 2);
                const int i = qi % T;
                const float2 cs = rope_s[i * (HD / 2) + e];
                q_s[qi * HD + e] = (x0[u] * cs.x - x1[u] * cs.y) * scale;
                q_s[qi * HD + e + HD / 2] = (x1[u] * cs.x + x0[u] * cs.y) * scale;
            }
        }
    }
    int nkeys = ncache;
    if (last) {
        // new K (RoPE) and V rows, rounded to bf16 exactly as they are cached, behind the cached keys
        for (int idx = tid; idx < T * (HD / 2); idx += AT_THREADS) {
            const int i = idx / (HD / 2), e = idx - i * (HD / 2);
            const float *row = a.zx + (size_t)(rowbase + i) * a.in_ld;
            const float2 cs = rope_s[idx];
            const float x0 = __ldcg(row + a.k_off + kh * HD + e), x1 = __ldcg(row + a.k_off + kh * HD + e + HD / 2);
            const __nv_bfloat16 k0 = __float2bfloat16_rn(x0 * cs.x - x1 * cs.y);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(x1 * cs.x + x0 * cs.y);
            const __nv_bfloat16 v0 = __float2bfloat16_rn(__ldcg(row + a.v_off + kh * HD + e));
            const __nv_bfloat16 v1 = __float2bfloat16_rn(__ldcg(row + a.v_off + kh * HD + e + HD / 2));
            const int j = ncache + i;
            K_s[j * HD + e] = k0; K_s[j * HD + e + HD / 2] = k1;
            V_s[j * HD + e] = v0; V_s[j * HD + e + HD / 2] = v1;
            Kb[(size_t)(len + i) * HD + e] = k0; Kb[(size_t)(len + i) * HD + e + HD / 2] = k1;
            Vb[(size_t)(len + i) * HD + e] = v0; Vb[(size_t)(len + i) * HD + e + HD / 2] = v1;
        }
        nkeys += T;
    }
    bool landed = true;
    if (ncache > 0) landed = mbar_wait(bar, 0);
    if (!__syncthreads_and(landed)) {             // a copy never landed: report it, contribute nothing, keep the barriers
        if (tid == 0) atomicCAS(a.status, 0, (int)HS_ERR_TIMEOUT);
        nkeys = 0;
    }

    // ---- scores: lane = key (tiles of 32), warp w takes query rows w, w + 4, ...
    for (int j0 = 0; j0 < nkeys; j0 += 32) {
        const int j = j0 + lane;
        const bool kvalid = j < nkeys;
        const uint4 *krow = reinterpret_cast<const uint4 *>(K_s + (size_t)min(j, nkeys - 1) * HD);
        for (int qb = warp; qb < GT; qb += AT_WARPS * 4) {
            // up to four query rows per pass: qb, qb + 4, qb + 8, qb + 12
            float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int c = 0; c < NC; ++c) {
                const int cc = (c + lane) & (NC - 1);          // rotated chunk order: conflict-free key reads
                const uint4 w = krow[cc];
                const float k0 = bf_lo(w.x), k1 = bf_hi(w.x), k2 = bf_lo(w.y), k3 = bf_hi(w.y);
                const float k4 = bf_lo(w.z), k5 = bf_hi(w.z), k6 = bf_lo(w.w), k7 = bf_hi(w.w);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int qi = qb + u * AT_WARPS;
                    if (qi < GT) {
                        const float4 qa = *reinterpret_cast<const float4 *>(q_s + qi * HD + cc * 8);
                        const float4 qc = *reinterpret_cast<const float4 *>(q_s + qi * HD + cc * 8 + 4);
                        d[u] = fmaf(k0, qa.x, fmaf(k1, qa.y, fmaf(k2, qa.z, fmaf(k3, qa.w, d[u]))));
                        d[u] = fmaf(k4, qc.x, fmaf(k5, qc.y, fmaf(k6, qc.z, fmaf(k7, qc.w, d[u]))));
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int qi = qb + u * AT_WARPS;
                if (qi < GT && kvalid) {
                    const int i = qi % T;
                    const bool masked = last && j >= ncache && (j - ncache) > i;     // causal among the new rows
                    p_s[qi * PST + j] = masked ? -INFINITY : d[u];
                }
            }
        }
    }
    __syncthreads();
    // ---- softmax statistics of the chunk: one warp per query row
    for (int qi = warp; qi < GT; qi += AT_WARPS) {
        float mx = -INFINITY;
        for (int j = lane; j < nkeys; j += 32) mx = fmaxf(mx, p_s[qi * PST + j]);
        mx = warp_max(mx);
        float sum = 0.f;
        for (int j = lane; j < nkeys; j += 32) {
            const float p = expf(p_s[qi * PST + j] - mx);        // expf(-inf) = 0 for masked keys
            p_s[qi * PST + j] = p;
            sum += p;
        }
        sum = warp_sum(sum);
        if (lane == 0) { ml_s[2 * qi] = mx; ml_s[2 * qi + 1] = sum; }
    }
    __syncthreads();
    // ---- acc = P V : thread = output dimension
    float acc[GTB];
#pragma unroll
    for (int qi = 0; qi < GTB; ++qi) acc[qi] = 0.f;
    if (tid < HD) {
        for (int j = 0; j < nkeys; ++j) {
            const float v = __bfloat162float(V_s[(size_t)j * HD + tid]);
#pragma unroll
            for (int qi = 0; qi < GTB; ++qi) if (qi < GT) acc[qi] = fmaf(p_s[qi * PST + j], v, acc[qi]);
        }
    }
    float *o_base = a.o + (size_t)rowbase * (a.qh * HD);
    // ---- combine the chunks of this cluster through distributed shared memory: every CTA leaves its partial
    //      (m, l, acc) in its own shared memory, rank r then sums output dims [r * DS, (r + 1) * DS) over all ranks
    constexpr int DS = HD / AT_CL;
    float *acc_s = q_s;                                      // [GT][HD]; the queries are no longer needed
    if (tid < HD) {
#pragma unroll
        for (int qi = 0; qi < GTB; ++qi) if (qi < GT) acc_s[qi * HD + tid] = acc[qi];
    }
    cluster.sync();
    float *mlr_s = p_s;                                      // [AT_CL][GT][2] copies of every rank's (m, l)
    float *wr_s = mlr_s + AT_CL * HS_MAX_GT * 2;             // [AT_CL][GT] merge weights
    float *Md_s = wr_s + AT_CL * HS_MAX_GT;                  // [GT][2] merged (M, den)
    for (int idx = tid; idx < AT_CL * GT * 2; idx += AT_THREADS) {
        const int r = idx / (GT * 2), rem = idx - r * (GT * 2);
        mlr_s[idx] = cluster.map_shared_rank(ml_s, r)[rem];
    }
    __syncthreads();
    if (tid < GT) {
        float M = -INFINITY;
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) M = fmaxf(M, mlr_s[(r * GT + tid) * 2]);
        float den = 0.f;
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) {
            const float mr = mlr_s[(r * GT + tid) * 2];
            const float w = mr == -INFINITY ? 0.f : expf(mr - M);
            wr_s[r * GT + tid] = w;
            den = fmaf(w, mlr_s[(r * GT + tid) * 2 + 1], den);
        }
        Md_s[2 * tid] = M; Md_s[2 * tid + 1] = den;
    }
    __syncthreads();
    const int nclus = (nsplit + AT_CL - 1) / AT_CL;
    const size_t pbase = ((size_t)b * a.kvh + kh) * a.nch;
    for (int idx = tid; idx < GT * DS; idx += AT_THREADS) {
        const int qi = idx / DS, d = crank * DS + (idx - qi * DS);
        float v[AT_CL];
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) v[r] = cluster.map_shared_rank(acc_s, r)[qi * HD + d];
        float sum = 0.f;
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) sum = fmaf(wr_s[r * GT + qi], v[r], sum);
        if (nclus == 1) {
            const int gq = qi / T, i = qi - gq * T;
            o_base[(size_t)i * (a.qh * HD) + (kh * G + gq) * HD + d] = sum / Md_s[2 * qi + 1];
        } else {
            a.part_acc[(pbase + cl) * HS_MAX_GT * HD + qi * HD + d] = sum;
        }
    }
    if (nclus > 1 && crank == 0 && tid < 2 * GT) a.part_ml[(pbase + cl) * HS_MAX_GT * 2 + tid] = Md_s[tid];
    cluster.sync();                                          // peers may still be reading this CTA's shared memory
    if (nclus == 1) return;
    // ---- several clusters: the CTA that arrives last merges the cluster partials in order
    __threadfence();
    __syncthreads();
    if (tid == 0) ticket_s = atomicAdd(a.counters + b * a.kvh + kh, 1);
    __syncthreads();
    if (ticket_s != nclus * AT_CL - 1) return;
    __threadfence();
    if (tid == 0) a.counters[b * a.kvh + kh] = 0;          // ready for the next launch
    const int nmerge = nclus;
    const float *pa0 = a.part_acc + pbase * HS_MAX_GT * HD;
    const float *pm0 = a.part_ml + pbase * HS_MAX_GT * 2;
    float *w_s = p_s;                                        // [GT][PST]: merge weights of PST chunks per pass
    for (int qi = warp; qi < GT; qi += AT_WARPS) {
        float M = -INFINITY;
        for (int c = lane; c < nmerge; c += 32) M = fmaxf(M, __ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
        M = warp_max(M);
        float den = 0.f;
        for (int c = lane; c < nmerge; c += 32) {
            const float2 mlv = __ldcg(reinterpret_cast<const float2 *>(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
            den = fmaf(expf(mlv.x - M), mlv.y, den);
        }
        den = warp_sum(den);
        if (lane == 0) { ml_s[2 * qi] = M; ml_s[2 * qi + 1] = den; }
    }
#pragma unroll
    for (int qi = 0; qi < GTB; ++qi) acc[qi] = 0.f;
    for (int cb = 0; cb < nmerge; cb += PST) {               // chunks in passes of PST
        const int nc = min(PST, nmerge - cb);
        __syncthreads();                                     // ml_s ready / previous pass done with w_s
        for (int idx = tid; idx < GT * nc; idx += AT_THREADS) {
            const int qi = idx / nc, c = idx - qi * nc;
            w_s[qi * PST + c] = expf(__ldcg(pm0 + ((size_t)(cb + c) * HS_MAX_GT + qi) * 2) - ml_s[2 * qi]);
        }
        __syncthreads();
        if (tid < HD) {
            constexpr int MB = 64 / GTB < 1 ? 1 : 64 / GTB;       // chunks whose partials are fetched together
            for (int c = 0; c < nc; c += MB) {
                float v[MB][GTB];
#pragma unroll
                for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                    for (int qi = 0; qi < GTB; ++qi)
                        v[mb][qi] = (c + mb < nc && qi < GT) ? __ldcg(pa0 + ((size_t)(cb + c + mb) * HS_MAX_GT + qi) * HD + tid) : 0.f;
#pragma unroll
                for (int mb = 0; mb < MB; ++mb)
#pragma unroll
                    for (int qi = 0; qi < GTB; ++qi)
                        if (c + mb < nc && qi < GT) acc[qi] = fmaf(w_s[qi * PST + c + mb], v[mb][qi], acc[qi]);
            }
        }
    }
    if (tid < HD) {
#pragma unroll
        for (int qi = 0; qi < GTB; ++qi)
            if (qi < GT) {
                const int gq = qi / T, i = qi - gq * T;
                o_base[(size_t)i * (a.qh * HD) + (kh * G + gq) * HD + tid] = acc[qi] / ml_s[2 * qi + 1];
            }
    }
}

template <int HD, int GTB>
cudaError_t launch_t(const AttnArgs &a, cudaStream_t s) {
    dim3 grid((a.nch + AT_CL - 1) / AT_CL * AT_CL, a.kvh, a.nb);
    return launch_pdl_cluster(attn_kernel<HD, GTB>, grid, dim3(AT_THREADS), AttnSmem<HD>::total(a.chunk), s, AT_CL, a);
}

template <int HD, int GTB>
cudaError_t configure_t() {
    cudaError_t e = cudaFuncSetAttribute(attn_kernel<HD, GTB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttnSmem<HD>::total(128));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel<HD, GTB>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    return e;
}

}  // namespace

cudaError_t configure_attn() {
    cudaError_t e = configure_t<128, 16>();
    if (e == cudaSuccess) e = configure_t<128, 32>();
    if (e == cudaSuccess) e = configure_t<128, 48>();
    if (e == cudaSuccess) e = configure_t<64, 16>();
    if (e == cudaSuccess) e = configure_t<64, 32>();
    if (e == cudaSuccess) e = configure_t<64, 48>();
    return e;
}

cudaError_t launch_attn(const AttnArgs &a, cudaStream_t s) {
    const int GT = (a.qh / a.kvh) * a.T;
    if (GT > HS_MAX_GT || (a.chunk != 32 && a.chunk != 64 && a.chunk != 128)) return cudaErrorInvalidValue;
    const int gtb = GT <= 16 ? 16 : GT <= 32 ? 32 : 48;
#define CASE(hd_, g_) if (a.hd == hd_ && gtb == g_) return launch_t<hd_, g_>(a, s)
    CASE(128, 16); CASE(128, 32); CASE(128, 48); CASE(64, 16); CASE(64, 32); CASE(64, 48);
#undef CASE
    return cudaErrorInvalidValue;
}

// Verify-mode attention: the T = k+1 new positions of a sequence attend over its KV cache plus the
// new rows themselves (causal among the new ones), grouped-query heads, split over the cache length.
//
// grid = (max splits, kv heads, sequences).  A block handles one split of `chunk` cached keys for
// the G*T query rows that share its KV head (G = q heads per KV head): K/V tiles of 32 keys are
// staged in shared memory as bf16, scores and the online softmax run in fp32, and the block writes
// either the final rows (single split) or an un-normalised partial (m, l, acc).  The block that
// covers the end of the cache also applies RoPE to the new K rows, appends the T new K/V rows
// (bf16) to the cache and attends to them from shared memory, so nothing written by this launch is
// read back from global memory by another block.  Partials are merged by whichever block arrives
// last (ticket counter, no spinning), always in split order, so the result is reproducible.
#include "hs_internal.h"
#include "hs_device.cuh"

namespace {
using namespace hsd;

constexpr int AT_THREADS = 128;
constexpr int KT = 32;                 // keys per tile

template <int HD>
__global__ void __launch_bounds__(AT_THREADS) attn_kernel(AttnArgs a) {
    constexpr int KSTR = HD + 8;       // padded bf16 row stride: 16-byte aligned, conflict-free 128-bit reads
    extern __shared__ __align__(16) unsigned char smraw[];
    const int G = a.qh / a.kvh, T = a.T, GT = G * T;
    float *q_s = reinterpret_cast<float *>(smraw);                         // [GT][HD] (RoPE'd, pre-scaled)
    float *p_s = q_s + HS_MAX_GT * HD;                                     // [GT][KT] scores -> probabilities
    float *m_s = p_s + HS_MAX_GT * KT;                                     // [GT] running max
    float *l_s = m_s + HS_MAX_GT;                                          // [GT] running sum
    float *c_s = l_s + HS_MAX_GT;                                          // [GT] rescale of this tile
    __nv_bfloat16 *K_s = reinterpret_cast<__nv_bfloat16 *>(c_s + HS_MAX_GT);   // [KT][KSTR]
    __nv_bfloat16 *V_s = K_s + KT * KSTR;                                  // [KT][KSTR]
    __nv_bfloat16 *Kn_s = V_s + KT * KSTR;                                 // [HS_MAX_T][KSTR] new rows
    __nv_bfloat16 *Vn_s = Kn_s + HS_MAX_T * KSTR;
    __shared__ int ticket_s;

    const int split = blockIdx.x, kh = blockIdx.y, lb = blockIdx.z, b = a.b0 + lb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait
    pdl_wait();
    const int len = __ldcg(a.kv_len + b);
    const int nch = max(1, (len + a.chunk - 1) / a.chunk);
    if (split >= nch) return;
    if (len + T > a.cap) {             // never write past the cache; the host reports the status word
        if (tid == 0 && split == 0 && kh == 0) atomicCAS(a.status, 0, (int)HS_ERR_CAPACITY);
        return;
    }
    const bool last = (split == nch - 1);
    const int rowbase = lb * T;
    const float scale = rsqrtf((float)HD);

    // ---- queries: RoPE at position len + i, pre-multiplied by 1/sqrt(hd)
    for (int idx = tid; idx < GT * (HD / 2); idx += AT_THREADS) {
        const int qi = idx / (HD / 2), e = idx - qi * (HD / 2);
        const int gq = qi / T, i = qi - gq * T;
        const float *src = a.zx + (size_t)(rowbase + i) * a.in_ld + a.q_off + (kh * G + gq) * HD;
        const float2 cs = a.rope[(size_t)(len + i) * (HD / 2) + e];
        const float x0 = __ldcg(src + e), x1 = __ldcg(src + e + HD / 2);
        q_s[qi * HD + e] = (x0 * cs.x - x1 * cs.y) * scale;
        q_s[qi * HD + e + HD / 2] = (x1 * cs.x + x0 * cs.y) * scale;
    }
    if (tid < GT) { m_s[tid] = -INFINITY; l_s[tid] = 0.f; }
    __nv_bfloat16 *Kb = a.Kc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    __nv_bfloat16 *Vb = a.Vc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    if (last) {
        // new K (RoPE) and V rows, rounded to bf16 exactly as they are cached
        for (int idx = tid; idx < T * (HD / 2); idx += AT_THREADS) {
            const int i = idx / (HD / 2), e = idx - i * (HD / 2);
            const float *row = a.zx + (size_t)(rowbase + i) * a.in_ld;
            const float2 cs = a.rope[(size_t)(len + i) * (HD / 2) + e];
            const float x0 = __ldcg(row + a.k_off + kh * HD + e), x1 = __ldcg(row + a.k_off + kh * HD + e + HD / 2);
            const __nv_bfloat16 k0 = __float2bfloat16_rn(x0 * cs.x - x1 * cs.y);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(x1 * cs.x + x0 * cs.y);
            const __nv_bfloat16 v0 = __float2bfloat16_rn(__ldcg(row + a.v_off + kh * HD + e));
            const __nv_bfloat16 v1 = __float2bfloat16_rn(__ldcg(row + a.v_off + kh * HD + e + HD / 2));
            Kn_s[i * KSTR + e] = k0; Kn_s[i * KSTR + e + HD / 2] = k1;
            Vn_s[i * KSTR + e] = v0; Vn_s[i * KSTR + e + HD / 2] = v1;
            Kb[(size_t)(len + i) * HD + e] = k0; Kb[(size_t)(len + i) * HD + e + HD / 2] = k1;
            Vb[(size_t)(len + i) * HD + e] = v0; Vb[(size_t)(len + i) * HD + e + HD / 2] = v1;
        }
    }
    float acc[HS_MAX_GT];              // thread tid < HD owns output dim tid of every query row
#pragma unroll
    for (int qi = 0; qi < HS_MAX_GT; ++qi) acc[qi] = 0.f;
    __syncthreads();

    const int c0 = split * a.chunk, c1 = min(len, c0 + a.chunk);
    const int ncache = max(0, c1 - c0);
    const int ntile_cache = (ncache + KT - 1) / KT;
    const int ntile = ntile_cache + (last ? 1 : 0);
    for (int t = 0; t < ntile; ++t) {
        const bool fresh = (t == ntile_cache);             // the tile of new rows (only when last)
        const int k0 = fresh ? len : c0 + t * KT;          // absolute index of the tile's first key
        const int nkeys = fresh ? T : min(KT, c1 - k0);
        // ---- stage the tile
        if (!fresh) {
            for (int idx = tid; idx < KT * (HD / 8); idx += AT_THREADS) {
                const int j = idx / (HD / 8), c = idx - j * (HD / 8);
                uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
                if (j < nkeys) {
                    kv = ldg_stream(Kb + (size_t)(k0 + j) * HD + 8 * c);
                    vv = ldg_stream(Vb + (size_t)(k0 + j) * HD + 8 * c);
                }
                *reinterpret_cast<uint4 *>(K_s + j * KSTR + 8 * c) = kv;
                *reinterpret_cast<uint4 *>(V_s + j * KSTR + 8 * c) = vv;
            }
            __syncthreads();
        }
        const __nv_bfloat16 *Kt_ = fresh ? Kn_s : K_s, *Vt_ = fresh ? Vn_s : V_s;
        // ---- scores: lane = key, warp w takes query rows w, w+4, ...
        for (int qi = warp; qi < GT; qi += AT_THREADS / 32) {
            float sc = -INFINITY;
            const int i = qi % T;
            if (lane < nkeys && (!fresh || lane <= i)) {     // causal among the new rows
                const uint4 *kr = reinterpret_cast<const uint4 *>(Kt_ + lane * KSTR);
                const float4 *qr = reinterpret_cast<const float4 *>(q_s + qi * HD);
                float d = 0.f;
#pragma unroll
                for (int c = 0; c < HD / 8; ++c) {
                    const uint4 w = kr[c];
                    const float4 qa = qr[2 * c], qb = qr[2 * c + 1];
                    d = fmaf(bf_lo(w.x), qa.x, d); d = fmaf(bf_hi(w.x), qa.y, d);
                    d = fmaf(bf_lo(w.y), qa.z, d); d = fmaf(bf_hi(w.y), qa.w, d);
                    d = fmaf(bf_lo(w.z), qb.x, d); d = fmaf(bf_hi(w.z), qb.y, d);
                    d = fmaf(bf_lo(w.w), qb.z, d); d = fmaf(bf_hi(w.w), qb.w, d);
                }
                sc = d;
            }
            const float m_old = m_s[qi];
            const float m_new = fmaxf(m_old, warp_max(sc));
            const float p = (sc == -INFINITY) ? 0.f : expf(sc - m_new);
            const float psum = warp_sum(p);
            p_s[qi * KT + lane] = p;
            if (lane == 0) {
                const float corr = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
                c_s[qi] = corr; m_s[qi] = m_new; l_s[qi] = l_s[qi] * corr + psum;
            }
        }
        __syncthreads();
        // ---- acc <- acc * corr + P V : thread = output dim
        if (tid < HD) {
#pragma unroll
            for (int qi = 0; qi < HS_MAX_GT; ++qi) if (qi < GT) acc[qi] *= c_s[qi];
            for (int j = 0; j < nkeys; ++j) {
                const float v = __bfloat162float(Vt_[j * KSTR + tid]);
#pragma unroll
                for (int qi = 0; qi < HS_MAX_GT; ++qi) if (qi < GT) acc[qi] = fmaf(p_s[qi * KT + j], v, acc[qi]);
            }
        }
        __syncthreads();
    }

    float *o_base = a.o + (size_t)rowbase * (a.qh * HD);
    if (nch == 1) {
        if (tid < HD) {
#pragma unroll
            for (int qi = 0; qi < HS_MAX_GT; ++qi)
                if (qi < GT) {
                    const int gq = qi / T, i = qi - gq * T;
                    o_base[(size_t)i * (a.qh * HD) + (kh * G + gq) * HD + tid] = acc[qi] / l_s[qi];
                }
        }
        return;
    }
    // ---- several splits: publish the partial, the last block to arrive merges in split order
    const size_t pbase = ((size_t)b * a.kvh + kh) * a.nch;
    float *pa = a.part_acc + (pbase + split) * HS_MAX_GT * HD;
    float *pm = a.part_ml + (pbase + split) * HS_MAX_GT * 2;
    if (tid < HD) {
#pragma unroll
        for (int qi = 0; qi < HS_MAX_GT; ++qi) if (qi < GT) pa[qi * HD + tid] = acc[qi];
    }
    if (tid < GT) { pm[2 * tid] = m_s[tid]; pm[2 * tid + 1] = l_s[tid]; }
    __threadfence();
    __syncthreads();
    if (tid == 0) ticket_s = atomicAdd(a.counters + b * a.kvh + kh, 1);
    __syncthreads();
    if (ticket_s != nch - 1) return;
    __threadfence();
    if (tid == 0) a.counters[b * a.kvh + kh] = 0;          // ready for the next launch
    const float *pa0 = a.part_acc + pbase * HS_MAX_GT * HD;
    const float *pm0 = a.part_ml + pbase * HS_MAX_GT * 2;
    if (tid < HD)
        for (int qi = 0; qi < GT; ++qi) {
            float M = -INFINITY;
            for (int c = 0; c < nch; ++c) M = fmaxf(M, __ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
            float num = 0.f, den = 0.f;
            for (int c = 0; c < nch; ++c) {
                const float w = expf(__ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2) - M);
                den = fmaf(w, __ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2 + 1), den);
                num = fmaf(w, __ldcg(pa0 + ((size_t)c * HS_MAX_GT + qi) * HD + tid), num);
            }
            const int gq = qi / T, i = qi - gq * T;
            o_base[(size_t)i * (a.qh * HD) + (kh * G + gq) * HD + tid] = num / den;
        }
}

template <int HD>
size_t attn_smem() {
    return (size_t)(HS_MAX_GT * HD + HS_MAX_GT * KT + 3 * HS_MAX_GT) * 4 +
           (size_t)(2 * KT + 2 * HS_MAX_T) * (HD + 8) * 2;
}

}  // namespace

cudaError_t configure_attn() {
    cudaError_t e = cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem<128>());
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem<64>());
    return e;
}

cudaError_t launch_attn(const AttnArgs &a, cudaStream_t s) {
    dim3 grid(a.nch, a.kvh, a.nb);
    if (a.hd == 128) return launch_pdl(attn_kernel<128>, grid, dim3(AT_THREADS), attn_smem<128>(), s, a);
    if (a.hd == 64) return launch_pdl(attn_kernel<64>, grid, dim3(AT_THREADS), attn_smem<64>(), s, a);
    return cudaErrorInvalidValue;
}

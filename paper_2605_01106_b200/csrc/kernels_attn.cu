// Verify-mode attention: the T = k+1 new positions of a sequence attend over its KV cache plus the
// new rows themselves (causal among the new ones), grouped-query heads, split over the cache length.
//
// grid = (key ranges rounded up to clusters of 8, kv heads, sequences); one CTA = a range of `tiles`
// tiles of CK cached keys each for the G*T query rows that share its KV head (G = q heads per KV head).
// Long caches at large batch use several tiles per CTA: the queries are staged and the partial combined
// once per range, and the tiles are folded into a running (max, sum, acc) - the online softmax.
//  * Before the programmatic-dependent-launch wait the CTA reads kv_len (written at least two kernels
//    earlier), starts the asynchronous copies of its first K and V tile into padded shared-memory rows
//    and fetches the RoPE rows of the new positions.  Later tiles are fetched while the previous one is
//    still in use: K for tile t+1 as soon as the scores of tile t are out, V after P V of tile t.
//  * After the wait it rotates and scales the queries; the CTA of the last chunk also rotates the T new
//    K rows, rounds K and V to bf16 exactly as they are cached, appends them to the cache and keeps them
//    in shared memory behind the cached keys, so nothing written by this launch is read back from
//    global memory by another block.
//  * Q K^T and P V run on the tensor cores (mma.sync m16n8k16, bf16 operands, fp32 accumulation).  K and
//    V are bf16 in the cache and enter exactly; the fp32 queries and probabilities are split into a
//    bf16 head and a bf16 remainder (two MMAs), which keeps the products exact to 2^-17 - the
//    comparison with the CPU oracle allows 1e-3 on states fed by this output.
//    Scores: a warp takes 16 keys at a time for all query rows; one softmax per tile (the whole tile is
//    resident); P V: a warp takes a quarter of the head dimension over all keys of the tile.
//  * The up to eight chunks of a cluster leave (m, l, acc) in their own shared memory and combine them
//    through distributed shared memory, rank r summing an eighth of the output dimensions.  Longer
//    caches span several clusters: each publishes one partial and the CTA that arrives last (ticket
//    counter, no spinning) merges them in order, so the result is reproducible.
#include "hs_internal.h"
#include "hs_device.cuh"
#include "ssm_body.cuh"
#include <cooperative_groups.h>

namespace {
using namespace hsd;
namespace cg = cooperative_groups;

constexpr int AT_THREADS = 128;
constexpr int AT_WARPS = 4;
constexpr int AT_CL = 8;               // CTAs (chunks) per thread-block cluster

struct AttnLayout {
    int kstr, keys, mrows, pstr, sstr;
    size_t k_off, v_off, q_off, s_off, p_off, ml_off, corr_off, new_off, rope_off, red_off, rx_off, total;
};
// shared-memory carve-up for head dim hd, chunk ck, gt query rows
__host__ __device__ inline AttnLayout attn_layout(int hd, int ck, int gt) {
    AttnLayout L;
    L.kstr = hd + 8;                       // padded bf16 row: 16-byte aligned, conflict-free ldmatrix
    L.keys = ck + 16;                      // cached keys + the new rows, rounded to the MMA k step
    L.mrows = (gt + 15) / 16 * 16;
    L.pstr = L.keys + 8;
    L.sstr = L.keys + 4;
    size_t o = 128;
    L.k_off = o; o += (size_t)L.keys * L.kstr * 2;
    L.v_off = o; o += (size_t)L.keys * L.kstr * 2;
    L.q_off = o; o += (size_t)2 * L.mrows * L.kstr * 2;       // bf16 head | remainder; later the fp32 partial acc
    L.s_off = o; o += (size_t)L.mrows * L.sstr * 4;           // raw scores fp32
    L.p_off = o; o += (size_t)2 * L.mrows * L.pstr * 2;       // probabilities: bf16 head | remainder
    L.ml_off = o; o += (size_t)HS_MAX_GT * 2 * 4;
    L.corr_off = o; o += (size_t)HS_MAX_GT * 4;
    L.new_off = o; o += (size_t)2 * HS_MAX_T * L.kstr * 2;    // the new K | V rows as they are cached
    L.rope_off = o; o += (size_t)HS_MAX_T * (hd / 2) * 8;
    L.red_off = o; o += (size_t)(AT_CL * HS_MAX_GT * 3 + HS_MAX_GT * 2) * 4;
    // what the peers of the cluster send: per source rank [gt][hd / AT_CL] partial outputs, then [gt][2] (max, sum)
    L.rx_off = o; o += (size_t)AT_CL * gt * (hd / AT_CL + 2) * 4;
    L.total = (o + 127) / 128 * 128;
    return L;
}

__device__ __forceinline__ void cp_async16(void *dst_smem, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(p)));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two floats rounded to bf16 (nearest even) and packed: lo in bits 0-15, hi in bits 16-31
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// x = head + remainder, both bf16 (round to nearest): exact to 2^-17 relative
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &h, __nv_bfloat16 &l) {
    h = __float2bfloat16_rn(x);
    l = __float2bfloat16_rn(x - __bfloat162float(h));
}

// MT: 16-row tiles of query rows (G*T <= 16 * MT).  The body takes its block coordinates as arguments
// (key range within the sequence, KV head, local sequence): it runs as a kernel of its own and as one of the
// two roles of the fused mixer + attention launch.  `split` must be the CTA's x index within a cluster-aligned
// row of the grid, so that split / 8 is the cluster and split % 8 the rank inside it.
template <int HD, int MT>
__device__ __forceinline__ void attn_body(const AttnArgs &a, const int split, const int kh, const int lb, unsigned char *smraw) {
    const int CK = a.chunk;
    const int G = a.qh / a.kvh, T = a.T, GT = G * T;
    const AttnLayout L = attn_layout(HD, CK, GT);
    const int KSTR = L.kstr, PSTR = L.pstr, SSTR = L.sstr;
    __nv_bfloat16 *K_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.k_off);         // [keys][KSTR]
    __nv_bfloat16 *V_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.v_off);
    __nv_bfloat16 *Qh_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.q_off);        // [mrows][KSTR] rotated, pre-scaled
    __nv_bfloat16 *Ql_s = Qh_s + (size_t)L.mrows * KSTR;
    float *s_s = reinterpret_cast<float *>(smraw + L.s_off);                         // [mrows][SSTR]
    __nv_bfloat16 *Ph_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.p_off);        // [mrows][PSTR]
    __nv_bfloat16 *Pl_s = Ph_s + (size_t)L.mrows * PSTR;
    float *ml_s = reinterpret_cast<float *>(smraw + L.ml_off);                       // [GT][2] running (max, sum)
    float *corr_s = reinterpret_cast<float *>(smraw + L.corr_off);                   // [GT] rescale of acc for this tile
    __nv_bfloat16 *Kn_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.new_off);      // [T][KSTR] new K rows (last CTA)
    __nv_bfloat16 *Vn_s = Kn_s + (size_t)HS_MAX_T * KSTR;
    float2 *rope_s = reinterpret_cast<float2 *>(smraw + L.rope_off);                 // [T][HD/2]
    float *red_s = reinterpret_cast<float *>(smraw + L.red_off);
    __shared__ int ticket_s;

    const int b = a.b0 + lb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t tinv = (65536u + T - 1) / T;      // x / T == (x * tinv) >> 16 for the small x used here
    pdl_trigger();          // the next kernel (out-projection) only streams weights before its own wait

    // ---- before the wait: kv_len, the first cached tile, the RoPE rows
    const int len = __ldcg(a.kv_len + b) + a.len_off;
    const int SPAN = CK * a.tiles;                // cached keys per CTA
    const int nsplit = max(1, (len + SPAN - 1) / SPAN);
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank(), cl = split / AT_CL;
    if (cl * AT_CL >= nsplit) return;             // the whole cluster is beyond the cache: nobody reaches a barrier
    // a CTA beyond the last range of a live cluster has no keys: it contributes (m, l) = (-inf, 0) and still
    // takes its share of the cluster's reduction
    const bool last = split == nsplit - 1;
    const int c0 = split * SPAN, rc = max(0, min(len, c0 + SPAN) - c0);
    const int ntile = last ? max(1, (rc + CK - 1) / CK) : (rc + CK - 1) / CK;
    if (len < 0 || len + T > a.cap) {             // never read or write outside the cache; the host reports the status word
        if (tid == 0 && split == 0 && kh == 0) atomicCAS(a.status, 0, len < 0 ? (int)HS_ERR_DEVICE : (int)HS_ERR_CAPACITY);
        return;
    }
    __nv_bfloat16 *Kb = a.Kc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    __nv_bfloat16 *Vb = a.Vc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    // asynchronous copy of the cached rows of tile t (one commit group per call, possibly empty)
    auto fetch = [&](__nv_bfloat16 *dst, const __nv_bfloat16 *src, int t) {
        const int n = t < ntile ? max(0, min(CK, rc - t * CK)) : 0;
        const __nv_bfloat16 *from = src + (size_t)(c0 + t * CK) * HD;
#pragma unroll 2
        for (int idx = tid; idx < n * (HD / 8); idx += AT_THREADS) {
            const int j = idx / (HD / 8), c = idx - j * (HD / 8);
            cp_async16(dst + (size_t)j * KSTR + 8 * c, from + (size_t)j * HD + 8 * c);
        }
        cp_async_commit();
    };
    fetch(K_s, Kb, 0);
    fetch(V_s, Vb, 0);
#pragma unroll 1
    for (int idx = tid; idx < T * (HD / 2); idx += AT_THREADS) {
        const int i = idx / (HD / 2), e = idx - i * (HD / 2);
        rope_s[idx] = a.rope[(size_t)(len + i) * (HD / 2) + e];
    }
    pdl_wait();
    __syncthreads();                        // rope_s complete

    // ---- queries: RoPE at position len + i, pre-multiplied by 1/sqrt(hd), split into bf16 head + remainder
    const int rowbase = lb * T;
    const float scale = rsqrtf((float)HD);
    // the CTA of the last key range also needs the raw k and v of the new positions: requested now, together with
    // the queries, so that both arrive after one trip to L2
    constexpr int NKV = (HS_MAX_T * (HD / 2) + AT_THREADS - 1) / AT_THREADS;
    float kraw[NKV][4];
    if (last) {
#pragma unroll
        for (int it = 0; it < NKV; ++it) {
            const int idx = tid + it * AT_THREADS;
            kraw[it][0] = kraw[it][1] = kraw[it][2] = kraw[it][3] = 0.f;
            if (idx < T * (HD / 2)) {
                const int i = idx / (HD / 2), e = idx - i * (HD / 2);
                const float *row = a.zx + (size_t)(rowbase + i) * a.in_ld;
                kraw[it][0] = __ldcg(row + a.k_off + kh * HD + e); kraw[it][1] = __ldcg(row + a.k_off + kh * HD + e + HD / 2);
                kraw[it][2] = __ldcg(row + a.v_off + kh * HD + e); kraw[it][3] = __ldcg(row + a.v_off + kh * HD + e + HD / 2);
            }
        }
    }
    {
        // thread = (rotation pair e, one of NH interleaved sets of query rows); four rows per round, whose loads
        // are all issued before the first use
        constexpr int HP = HD / 2, NH = AT_THREADS / HP;      // 64 pairs x 2 sets (hd 128) or 32 x 4 (hd 64)
        const int e = tid % HP, part = tid / HP;
#pragma unroll 1
        for (int q0 = part; q0 < GT; q0 += 4 * NH) {
            float x0[4], x1[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int qi = q0 + u * NH;
                x0[u] = x1[u] = 0.f;
                if (qi < GT) {
                    const int gq = (int)((qi * tinv) >> 16);
                    const float *src = a.zx + (size_t)(rowbase + qi - gq * T) * a.in_ld + a.q_off + (kh * G + gq) * HD;
                    x0[u] = __ldcg(src + e); x1[u] = __ldcg(src + e + HP);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int qi = q0 + u * NH;
                if (qi < GT) {
                    const float2 cs = rope_s[(qi - (int)((qi * tinv) >> 16) * T) * HP + e];
                    __nv_bfloat16 h, l;
                    split_bf16((x0[u] * cs.x - x1[u] * cs.y) * scale, h, l);
                    Qh_s[qi * KSTR + e] = h; Ql_s[qi * KSTR + e] = l;
                    split_bf16((x1[u] * cs.x + x0[u] * cs.y) * scale, h, l);
                    Qh_s[qi * KSTR + e + HP] = h; Ql_s[qi * KSTR + e + HP] = l;
                }
            }
        }
    }
    if (last) {
        // new K (RoPE) and V rows, rounded to bf16 exactly as they are cached: appended to the cache and kept
        // aside; they join the last tile behind its cached keys
#pragma unroll
        for (int it = 0; it < NKV; ++it) {
            const int idx = tid + it * AT_THREADS;
            if (idx >= T * (HD / 2)) break;
            const int i = idx / (HD / 2), e = idx - i * (HD / 2);
            const float2 cs = rope_s[idx];
            const float x0 = kraw[it][0], x1 = kraw[it][1];
            const __nv_bfloat16 k0 = __float2bfloat16_rn(x0 * cs.x - x1 * cs.y);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(x1 * cs.x + x0 * cs.y);
            const __nv_bfloat16 v0 = __float2bfloat16_rn(kraw[it][2]);
            const __nv_bfloat16 v1 = __float2bfloat16_rn(kraw[it][3]);
            Kn_s[i * KSTR + e] = k0; Kn_s[i * KSTR + e + HD / 2] = k1;
            Vn_s[i * KSTR + e] = v0; Vn_s[i * KSTR + e + HD / 2] = v1;
            Kb[(size_t)(len + i) * HD + e] = k0; Kb[(size_t)(len + i) * HD + e + HD / 2] = k1;
            Vb[(size_t)(len + i) * HD + e] = v0; Vb[(size_t)(len + i) * HD + e + HD / 2] = v1;
        }
    }
    if (tid < GT) { ml_s[2 * tid] = -INFINITY; ml_s[2 * tid + 1] = 0.f; }
    const int g8 = lane >> 2, t4 = lane & 3;
    constexpr int DW = HD / AT_WARPS, NTW = DW / 8;
    float O[MT][NTW][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) { O[mt][nt][0] = O[mt][nt][1] = O[mt][nt][2] = O[mt][nt][3] = 0.f; }
    __syncthreads();                        // queries, new rows, running stats in place

#pragma unroll 1
    for (int t = 0; t < ntile; ++t) {
        const int ncache = max(0, min(CK, rc - t * CK));
        const bool lastt = last && t == ntile - 1;     // the tile that also holds the new rows
        const int nkeys = ncache + (lastt ? T : 0);
        const int nkp = (nkeys + 15) & ~15;            // keys rounded to the MMA k step
        if (lastt) {
#pragma unroll 1
            for (int idx = tid; idx < T * (HD / 8); idx += AT_THREADS) {
                const int i = idx / (HD / 8), c = idx - i * (HD / 8);
                *reinterpret_cast<uint4 *>(K_s + (size_t)(ncache + i) * KSTR + 8 * c) = *reinterpret_cast<const uint4 *>(Kn_s + (size_t)i * KSTR + 8 * c);
                *reinterpret_cast<uint4 *>(V_s + (size_t)(ncache + i) * KSTR + 8 * c) = *reinterpret_cast<const uint4 *>(Vn_s + (size_t)i * KSTR + 8 * c);
            }
            // V rows of the padding keys must be finite: their probabilities are zero, and 0 * NaN is not
#pragma unroll 1
            for (int idx = tid; idx < (nkp - nkeys) * (HD / 8); idx += AT_THREADS) {
                const int j = nkeys + idx / (HD / 8), c = idx % (HD / 8);
                *reinterpret_cast<uint4 *>(V_s + (size_t)j * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
            }
        }
        cp_async_wait_but_one();            // K of this tile has landed (V may still be in flight)
        __syncthreads();

        // ---- scores S = Q K^T on the tensor cores: a warp takes 16 keys at a time for all query rows
#pragma unroll 1
        for (int grp = warp; grp * 16 < nkp; grp += AT_WARPS) {
            const int kb = grp * 16;
            float S[MT][2][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) { S[mt][nt][0] = S[mt][nt][1] = S[mt][nt][2] = S[mt][nt][3] = 0.f; }
#pragma unroll 4
            for (int ks = 0; ks < HD / 16; ++ks) {
                uint32_t bk[4];
                ldsm_x4(bk, K_s + (size_t)(kb + (lane & 7) + (lane >> 4) * 8) * KSTR + ks * 16 + ((lane >> 3) & 1) * 8);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    uint32_t ah[4], al[4];
                    const size_t qo = (size_t)(mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * KSTR + ks * 16 + (lane >> 4) * 8;
                    ldsm_x4(ah, Qh_s + qo);
                    ldsm_x4(al, Ql_s + qo);
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) mma_bf16(S[mt][nt], ah, bk[nt * 2], bk[nt * 2 + 1]);
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) mma_bf16(S[mt][nt], al, bk[nt * 2], bk[nt * 2 + 1]);
                }
            }
            // raw scores to shared memory; keys beyond the tile and, among the new rows, later positions are masked
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int row = mt * 16 + g8 + (e >> 1) * 8, key = kb + nt * 8 + 2 * t4 + (e & 1);
                        if (row < GT) {
                            const bool masked = key >= nkeys || (lastt && key >= ncache && (key - ncache) > (row - (int)((row * tinv) >> 16) * T));
                            s_s[row * SSTR + key] = masked ? -INFINITY : S[mt][nt][e];
                        }
                    }
        }
        __syncthreads();
        fetch(K_s, Kb, t + 1);              // the K buffer is free: next tile's keys arrive during softmax and P V
        // ---- softmax of the tile folded into the running (max, sum): eight lanes per query row, sixteen rows
        //      per pass; probabilities as bf16 head + remainder
        // lanes per query row: as many as the block has for GT rows (a power of two up to 32), so that a few rows
        // (small k) are not left to a fraction of one warp
        const int LPR = GT * 32 <= AT_THREADS ? 32 : GT * 16 <= AT_THREADS ? 16 : GT * 8 <= AT_THREADS ? 8 : 4;
        const int lsh = LPR == 32 ? 5 : LPR == 16 ? 4 : LPR == 8 ? 3 : 2;
#pragma unroll 1
        for (int q0 = 0; q0 < GT; q0 += AT_THREADS / LPR) {
            const int qi = q0 + (tid >> lsh), sub = tid & (LPR - 1);
            const bool rv = qi < GT;
            const float m_old = rv ? ml_s[2 * qi] : -INFINITY, l_old = rv ? ml_s[2 * qi + 1] : 0.f;
            float mx = m_old;
            if (rv)
#pragma unroll 4
                for (int j = sub; j < nkp; j += LPR) mx = fmaxf(mx, s_s[qi * SSTR + j]);
#pragma unroll 1
            for (int o = LPR / 2; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float sum = 0.f;
            if (rv)
#pragma unroll 2
                for (int j = sub; j < nkp; j += LPR) {
                    const float sv = s_s[qi * SSTR + j];
                    const float p = sv == -INFINITY ? 0.f : __expf(sv - mx);
                    __nv_bfloat16 h, l;
                    split_bf16(p, h, l);
                    Ph_s[qi * PSTR + j] = h; Pl_s[qi * PSTR + j] = l;
                    sum += p;
                }
#pragma unroll 1
            for (int o = LPR / 2; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (rv && sub == 0) {
                const float corr = m_old == -INFINITY ? 0.f : __expf(m_old - mx);
                ml_s[2 * qi] = mx; ml_s[2 * qi + 1] = fmaf(l_old, corr, sum);
                corr_s[qi] = corr;
            }
        }
        cp_async_wait_but_one();            // V of this tile has landed (the next K may still be in flight)
        __syncthreads();
        // ---- acc = acc * corr + P V on the tensor cores: a warp takes a quarter of the head dimension
        if (t > 0) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const int r0 = mt * 16 + g8, r1 = r0 + 8;
                const float c0r = r0 < GT ? corr_s[r0] : 1.f, c1r = r1 < GT ? corr_s[r1] : 1.f;
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt) { O[mt][nt][0] *= c0r; O[mt][nt][1] *= c0r; O[mt][nt][2] *= c1r; O[mt][nt][3] *= c1r; }
            }
        }
#pragma unroll 2
        for (int kk = 0; kk < nkp / 16; ++kk) {
            uint32_t bv[NTW / 2][4];
#pragma unroll
            for (int p = 0; p < NTW / 2; ++p)
                ldsm_x4_t(bv[p], V_s + (size_t)(kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * KSTR + warp * DW + p * 16 + (lane >> 4) * 8);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                uint32_t ah[4], al[4];
                const size_t po = (size_t)(mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PSTR + kk * 16 + (lane >> 4) * 8;
                ldsm_x4(ah, Ph_s + po);
                ldsm_x4(al, Pl_s + po);
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt) mma_bf16(O[mt][nt], ah, bv[nt >> 1][(nt & 1) * 2], bv[nt >> 1][(nt & 1) * 2 + 1]);
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt) mma_bf16(O[mt][nt], al, bv[nt >> 1][(nt & 1) * 2], bv[nt >> 1][(nt & 1) * 2 + 1]);
            }
        }
        __syncthreads();                    // everybody is done with V, P and the scores of this tile
        fetch(V_s, Vb, t + 1);
    }
    cp_async_wait_all();                    // only empty groups can be left
    // ---- combine the key ranges of this cluster.  Rank r finishes the output dimensions [r * DS, (r + 1) * DS):
    //      every CTA that holds keys stores, straight from its accumulator registers, the slice each peer finishes
    //      into that peer's shared memory (plus its running max and sum), the cluster meets at ONE barrier, and every
    //      rank merges what it received - in rank order, so the result does not depend on timing.  Nothing is read
    //      from a peer after the barrier, so a CTA may exit as soon as it is done.
    constexpr int DS = HD / AT_CL;
    float *rx_acc = reinterpret_cast<float *>(smraw + L.rx_off);          // [source rank][GT][DS]
    float *rx_ml = rx_acc + (size_t)AT_CL * GT * DS;                       // [source rank][GT][2]
    const int nlive = min(AT_CL, nsplit - cl * AT_CL);                     // ranks of this cluster that hold keys
    if (crank < nlive) {
        const uint32_t acc_a = smem_u32(rx_acc) + (uint32_t)crank * GT * DS * 4;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int row = mt * 16 + g8 + hh * 8, d = warp * DW + nt * 8 + 2 * t4;
                    if (row < GT)
                        dsmem_st_v2(dsmem_addr(acc_a + (uint32_t)(row * DS + (d % DS)) * 4, (uint32_t)(d / DS)), O[mt][nt][2 * hh], O[mt][nt][2 * hh + 1]);
                }
        const uint32_t ml_a = smem_u32(rx_ml) + (uint32_t)crank * GT * 2 * 4;
#pragma unroll 1
        for (int idx = tid; idx < GT * AT_CL; idx += AT_THREADS) {
            const int dest = idx & (AT_CL - 1), qi = idx >> 3;
            dsmem_st_v2(dsmem_addr(ml_a + (uint32_t)qi * 8, (uint32_t)dest), ml_s[2 * qi], ml_s[2 * qi + 1]);
        }
    }
    float *o_base = a.o + (size_t)rowbase * (a.qh * HD);
    cluster_arrive(); cluster_wait();
    const int nclus = (nsplit + AT_CL - 1) / AT_CL;
    const size_t pbase = ((size_t)b * a.kvh + kh) * a.nch;
    float *Md_s = red_s;                                     // [GT][2] merged (M, den), for the cluster partial
    constexpr int DV = DS / 4;                               // a thread takes four output dimensions of one query row
#pragma unroll 1
    for (int idx = tid; idx < GT * DV; idx += AT_THREADS) {
        const int qi = idx / DV, dd = (idx - qi * DV) * 4, d = crank * DS + dd;
        float2 mlr[AT_CL];
        float4 v[AT_CL];
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) {
            mlr[r] = make_float2(-INFINITY, 0.f); v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < nlive) {
                mlr[r] = *reinterpret_cast<const float2 *>(rx_ml + ((size_t)r * GT + qi) * 2);
                v[r] = *reinterpret_cast<const float4 *>(rx_acc + ((size_t)r * GT + qi) * DS + dd);
            }
        }
        float M = -INFINITY;
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) M = fmaxf(M, mlr[r].x);
        float den = 0.f;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r = 0; r < AT_CL; ++r) {
            const float w = mlr[r].x == -INFINITY ? 0.f : __expf(mlr[r].x - M);
            den = fmaf(w, mlr[r].y, den);
            sum.x = fmaf(w, v[r].x, sum.x); sum.y = fmaf(w, v[r].y, sum.y);
            sum.z = fmaf(w, v[r].z, sum.z); sum.w = fmaf(w, v[r].w, sum.w);
        }
        if (nclus == 1) {
            const int gq = (int)((qi * tinv) >> 16), i = qi - gq * T;
            const float inv = 1.0f / den;
            *reinterpret_cast<float4 *>(o_base + (size_t)i * (a.qh * HD) + (kh * G + gq) * HD + d) =
                make_float4(sum.x * inv, sum.y * inv, sum.z * inv, sum.w * inv);
        } else {
            *reinterpret_cast<float4 *>(a.part_acc + (pbase + cl) * HS_MAX_GT * HD + qi * HD + d) = sum;
            if (crank == 0 && dd == 0) { Md_s[2 * qi] = M; Md_s[2 * qi + 1] = den; }
        }
    }
    if (nclus > 1) __syncthreads();
    if (nclus > 1 && crank == 0 && tid < 2 * GT) a.part_ml[(pbase + cl) * HS_MAX_GT * 2 + tid] = Md_s[tid];
    if (nclus == 1) return;
    // ---- several clusters: the CTA that arrives last merges the cluster partials in order
    __threadfence();
    __syncthreads();
    if (tid == 0) ticket_s = atomicAdd(a.counters + b * a.kvh + kh, 1);
    __syncthreads();
    if (ticket_s != nclus * AT_CL - 1) return;
    __threadfence();
    if (tid == 0) a.counters[b * a.kvh + kh] = 0;          // ready for the next launch
    constexpr int GTB = MT * 16;
    const float *pa0 = a.part_acc + pbase * HS_MAX_GT * HD;
    const float *pm0 = a.part_ml + pbase * HS_MAX_GT * 2;
    float *w_s = s_s;                                        // [GT][SSTR]: merge weights of SSTR clusters per pass
    for (int qi = warp; qi < GT; qi += AT_WARPS) {
        float M = -INFINITY;
        for (int c = lane; c < nclus; c += 32) M = fmaxf(M, __ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
        M = warp_max(M);
        float den = 0.f;
        for (int c = lane; c < nclus; c += 32) {
            const float2 mlv = __ldcg(reinterpret_cast<const float2 *>(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
            den = fmaf(__expf(mlv.x - M), mlv.y, den);
        }
        den = warp_sum(den);
        if (lane == 0) { ml_s[2 * qi] = M; ml_s[2 * qi + 1] = den; }
    }
    float acc[GTB];
#pragma unroll
    for (int qi = 0; qi < GTB; ++qi) acc[qi] = 0.f;
    for (int cb = 0; cb < nclus; cb += SSTR) {               // clusters in passes of SSTR
        const int nc = min(SSTR, nclus - cb);
        __syncthreads();                                     // ml_s ready / previous pass done with w_s
        for (int idx = tid; idx < GT * nc; idx += AT_THREADS) {
            const int qi = idx / nc, c = idx - qi * nc;
            w_s[qi * SSTR + c] = __expf(__ldcg(pm0 + ((size_t)(cb + c) * HS_MAX_GT + qi) * 2) - ml_s[2 * qi]);
        }
        __syncthreads();
        if (tid < HD) {
            constexpr int MB = 64 / GTB < 1 ? 1 : 64 / GTB;       // clusters whose partials are fetched together
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
                        if (c + mb < nc && qi < GT) acc[qi] = fmaf(w_s[qi * SSTR + c + mb], v[mb][qi], acc[qi]);
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


// ------------------------------------------------------------------------------------------------
// Short caches and few query rows (G*T <= 16, the whole cache within one cluster of eight CTAs): the
// latency-lean form.  A CTA holds its whole key range (up to 256 cached keys plus the new rows) in shared
// memory, fetched before the dependency wait.  After the queries are staged there is no block-wide
// synchronisation any more: every warp takes 16 keys at a time, computes the scores on the tensor cores,
// keeps the probabilities in registers (the accumulator layout of the score tile is the operand layout of
// the P V product), runs its own running softmax over its key groups and accumulates its own partial output
// over the full head dimension.  Each warp then stores, straight from registers, the slice of its partial that
// each rank of the cluster finishes into that rank's shared memory, the cluster meets at one barrier, and
// every rank merges the 4 x 8 warp partials of its output dimensions in a fixed order.
struct AttnSmallLayout { int kstr, keys; size_t k_off, v_off, q_off, rope_off, rx_off, total; };
__host__ __device__ inline AttnSmallLayout attn_small_layout(int hd, int ck, int gt) {
    AttnSmallLayout L;
    L.kstr = hd + 8;
    L.keys = ck + 16;                      // cached keys + the new rows, rounded to the MMA k step
    size_t o = 128;
    L.k_off = o; o += (size_t)L.keys * L.kstr * 2;
    L.v_off = o; o += (size_t)L.keys * L.kstr * 2;
    L.q_off = o; o += (size_t)2 * 16 * L.kstr * 2;              // 16 query rows: bf16 head | remainder
    L.rope_off = o; o += (size_t)HS_MAX_T * (hd / 2) * 8;
    L.rx_off = o; o += (size_t)AT_CL * AT_WARPS * gt * (hd / AT_CL + 2) * 4;   // per source warp: [gt][hd/8] partials, [gt][2] (max, sum)
    L.total = (o + 127) / 128 * 128;
    return L;
}
constexpr int AT_SMALL_MAXCHUNK = 256;

template <int HD>
__device__ __forceinline__ void attn_small_body(const AttnArgs &a, const int split, const int kh, const int lb, unsigned char *smraw) {
    const int CK = a.chunk;                        // cached keys per CTA: a multiple of 16 up to 256
    const int G = a.qh / a.kvh, T = a.T, GT = G * T;
    const AttnSmallLayout L = attn_small_layout(HD, CK, GT);
    const int KSTR = L.kstr;
    __nv_bfloat16 *K_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.k_off);         // [keys][KSTR]
    __nv_bfloat16 *V_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.v_off);
    __nv_bfloat16 *Qh_s = reinterpret_cast<__nv_bfloat16 *>(smraw + L.q_off);        // [16][KSTR] rotated, pre-scaled
    __nv_bfloat16 *Ql_s = Qh_s + (size_t)16 * KSTR;
    float2 *rope_s = reinterpret_cast<float2 *>(smraw + L.rope_off);                 // [T][HD/2]
    constexpr int DS = HD / AT_CL, NSRC = AT_CL * AT_WARPS;
    float *rx_acc = reinterpret_cast<float *>(smraw + L.rx_off);                     // [source warp][GT][DS]
    float *rx_ml = rx_acc + (size_t)NSRC * GT * DS;                                  // [source warp][GT][2]

    const int b = a.b0 + lb;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t tinv = (65536u + T - 1) / T;      // x / T == (x * tinv) >> 16 for the small x used here
    pdl_trigger();

    // ---- before the wait: kv_len, the whole key range of this CTA, the RoPE rows
    const int len = __ldcg(a.kv_len + b) + a.len_off;
    const int nsplit = max(1, (len + CK - 1) / CK);
    if (len < 0 || len + T > a.cap || nsplit > AT_CL) {      // never write past the cache; a cache longer than the host's bound is a host error
        if (tid == 0 && split == 0 && kh == 0) atomicCAS(a.status, 0, (len >= 0 && len + T > a.cap) ? (int)HS_ERR_CAPACITY : (int)HS_ERR_DEVICE);
        return;
    }
    const int crank = split;                      // the grid has exactly one cluster along x
    const bool live = split < nsplit, last = split == nsplit - 1;
    const int c0 = split * CK, rc = live ? min(len, c0 + CK) - c0 : 0;
    __nv_bfloat16 *Kb = a.Kc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    __nv_bfloat16 *Vb = a.Vc + ((size_t)b * a.kvh + kh) * a.cap * HD;
#pragma unroll 2
    for (int idx = tid; idx < rc * (HD / 8); idx += AT_THREADS) {
        const int j = idx / (HD / 8), c = idx - j * (HD / 8);
        cp_async16(K_s + (size_t)j * KSTR + 8 * c, Kb + (size_t)(c0 + j) * HD + 8 * c);
    }
#pragma unroll 2
    for (int idx = tid; idx < rc * (HD / 8); idx += AT_THREADS) {
        const int j = idx / (HD / 8), c = idx - j * (HD / 8);
        cp_async16(V_s + (size_t)j * KSTR + 8 * c, Vb + (size_t)(c0 + j) * HD + 8 * c);
    }
    cp_async_commit();
#pragma unroll 1
    for (int idx = tid; idx < T * (HD / 2); idx += AT_THREADS) {
        const int i = idx / (HD / 2), e = idx - i * (HD / 2);
        rope_s[idx] = a.rope[(size_t)(len + i) * (HD / 2) + e];
    }
    // query rows that do not exist are zero (their results are never stored)
#pragma unroll 1
    for (int idx = tid; idx < (16 - GT) * (HD / 8); idx += AT_THREADS) {
        const int r = GT + idx / (HD / 8), c = idx % (HD / 8);
        *reinterpret_cast<uint4 *>(Qh_s + (size_t)r * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(Ql_s + (size_t)r * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
    }
    const int rowbase = lb * T;
    const float scale = rsqrtf((float)HD);
    const int nkeys = rc + (last ? T : 0);
    const int nkp = (nkeys + 15) & ~15;
    pdl_wait();
    __syncthreads();                        // rope_s complete

    // ---- after the wait: one trip to L2 for the queries and (last key range) the raw k, v of the new positions
    constexpr int NKV = (HS_MAX_T * (HD / 2) + AT_THREADS - 1) / AT_THREADS;
    float kraw[NKV][4];
    if (last) {
#pragma unroll
        for (int it = 0; it < NKV; ++it) {
            const int idx = tid + it * AT_THREADS;
            kraw[it][0] = kraw[it][1] = kraw[it][2] = kraw[it][3] = 0.f;
            if (idx < T * (HD / 2)) {
                const int i = idx / (HD / 2), e = idx - i * (HD / 2);
                const float *row = a.zx + (size_t)(rowbase + i) * a.in_ld;
                kraw[it][0] = __ldcg(row + a.k_off + kh * HD + e); kraw[it][1] = __ldcg(row + a.k_off + kh * HD + e + HD / 2);
                kraw[it][2] = __ldcg(row + a.v_off + kh * HD + e); kraw[it][3] = __ldcg(row + a.v_off + kh * HD + e + HD / 2);
            }
        }
    }
    if (live) {
        // thread = (rotation pair e, one of NH interleaved sets of query rows); every load is issued before the first use
        constexpr int HP = HD / 2, NH = AT_THREADS / HP, U = 16 / NH;
        const int e = tid % HP, part = tid / HP;
        float x0[U], x1[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int qi = part + u * NH;
            x0[u] = x1[u] = 0.f;
            if (qi < GT) {
                const int gq = (int)((qi * tinv) >> 16);
                const float *src = a.zx + (size_t)(rowbase + qi - gq * T) * a.in_ld + a.q_off + (kh * G + gq) * HD;
                x0[u] = __ldcg(src + e); x1[u] = __ldcg(src + e + HP);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int qi = part + u * NH;
            if (qi < GT) {
                const float2 cs = rope_s[(qi - (int)((qi * tinv) >> 16) * T) * HP + e];
                __nv_bfloat16 h, l;
                split_bf16((x0[u] * cs.x - x1[u] * cs.y) * scale, h, l);
                Qh_s[qi * KSTR + e] = h; Ql_s[qi * KSTR + e] = l;
                split_bf16((x1[u] * cs.x + x0[u] * cs.y) * scale, h, l);
                Qh_s[qi * KSTR + e + HP] = h; Ql_s[qi * KSTR + e + HP] = l;
            }
        }
    }
    if (last) {
        // new K (RoPE) and V rows, rounded to bf16 exactly as they are cached: appended to the cache and placed behind
        // the cached keys of this range
#pragma unroll
        for (int it = 0; it < NKV; ++it) {
            const int idx = tid + it * AT_THREADS;
            if (idx >= T * (HD / 2)) break;
            const int i = idx / (HD / 2), e = idx - i * (HD / 2);
            const float2 cs = rope_s[idx];
            const float x0 = kraw[it][0], x1 = kraw[it][1];
            const __nv_bfloat16 k0 = __float2bfloat16_rn(x0 * cs.x - x1 * cs.y);
            const __nv_bfloat16 k1 = __float2bfloat16_rn(x1 * cs.x + x0 * cs.y);
            const __nv_bfloat16 v0 = __float2bfloat16_rn(kraw[it][2]);
            const __nv_bfloat16 v1 = __float2bfloat16_rn(kraw[it][3]);
            K_s[(size_t)(rc + i) * KSTR + e] = k0; K_s[(size_t)(rc + i) * KSTR + e + HD / 2] = k1;
            V_s[(size_t)(rc + i) * KSTR + e] = v0; V_s[(size_t)(rc + i) * KSTR + e + HD / 2] = v1;
            Kb[(size_t)(len + i) * HD + e] = k0; Kb[(size_t)(len + i) * HD + e + HD / 2] = k1;
            Vb[(size_t)(len + i) * HD + e] = v0; Vb[(size_t)(len + i) * HD + e + HD / 2] = v1;
        }
    }
    // V rows of the padding keys must be finite: their probabilities are zero, and 0 * NaN is not
#pragma unroll 1
    for (int idx = tid; idx < (nkp - nkeys) * (HD / 8); idx += AT_THREADS) {
        const int j = nkeys + idx / (HD / 8), c = idx % (HD / 8);
        *reinterpret_cast<uint4 *>(V_s + (size_t)j * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
    }
    cp_async_wait_all();
    __syncthreads();                        // keys, values, queries in place: the last block-wide barrier

    // ---- per warp: 16 keys at a time, probabilities in registers, running softmax, partial output over all of HD
    const int g8 = lane >> 2, t4 = lane & 3;
    constexpr int NT = HD / 8;
    float O[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { O[nt][0] = O[nt][1] = O[nt][2] = O[nt][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};      // rows g8 and g8 + 8
    const int ti0 = g8 - (int)((g8 * tinv) >> 16) * T, ti1 = (g8 + 8) - (int)(((g8 + 8) * tinv) >> 16) * T;   // position index of the two rows
#pragma unroll 1
    for (int kb = warp * 16; kb < nkp; kb += AT_WARPS * 16) {
        // scores: the k steps feed four accumulator sets in turn, so that a chain of dependent MMAs is 4 long, not 16
        float Sp[4][2][4];
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) { Sp[c][nt][0] = Sp[c][nt][1] = Sp[c][nt][2] = Sp[c][nt][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            uint32_t bk[4], ah[4], al[4];
            ldsm_x4(bk, K_s + (size_t)(kb + (lane & 7) + (lane >> 4) * 8) * KSTR + ks * 16 + ((lane >> 3) & 1) * 8);
            const size_t qo = (size_t)((lane & 7) + ((lane >> 3) & 1) * 8) * KSTR + ks * 16 + (lane >> 4) * 8;
            ldsm_x4(ah, Qh_s + qo);
            ldsm_x4(al, Ql_s + qo);
            mma_bf16(Sp[(2 * ks) & 3][0], ah, bk[0], bk[1]); mma_bf16(Sp[(2 * ks) & 3][1], ah, bk[2], bk[3]);
            mma_bf16(Sp[(2 * ks + 1) & 3][0], al, bk[0], bk[1]); mma_bf16(Sp[(2 * ks + 1) & 3][1], al, bk[2], bk[3]);
        }
        float S[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) S[nt][e] = (Sp[0][nt][e] + Sp[1][nt][e]) + (Sp[2][nt][e] + Sp[3][nt][e]);
        // masks: keys beyond the range and, among the new rows, later positions
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = kb + nt * 8 + 2 * t4 + (e & 1), ti = (e >> 1) ? ti1 : ti0;
                if (key >= nkeys || (last && key >= rc && key - rc > ti)) S[nt][e] = -INFINITY;
                mx[e >> 1] = fmaxf(mx[e >> 1], S[nt][e]);
            }
        uint32_t ph[4], pl[4];
        float corr[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float mnew = fmaxf(m_run[r], mx[r]);
            const float muse = mnew == -INFINITY ? 0.f : mnew;         // a row that has seen no key yet: everything stays zero
            corr[r] = __expf(m_run[r] - muse);                        // exp(-inf) = 0 on the first group
            m_run[r] = mnew;
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                const float p0 = __expf(S[nt][2 * r] - muse), p1 = __expf(S[nt][2 * r + 1] - muse);
                sum += p0 + p1;
                __nv_bfloat16 h0, l0, h1, l1;
                split_bf16(p0, h0, l0); split_bf16(p1, h1, l1);
                // A fragment of P (16 rows x 16 keys): register r + 2 * nt holds row g8 + 8 r, keys 8 nt + 2 t4, + 1
                ph[r + 2 * nt] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                pl[r + 2 * nt] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
            }
            l_run[r] = fmaf(l_run[r], corr[r], sum);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { O[nt][0] *= corr[0]; O[nt][1] *= corr[0]; O[nt][2] *= corr[1]; O[nt][3] *= corr[1]; }
#pragma unroll
        for (int p = 0; p < NT / 2; ++p) {
            uint32_t bv[4];
            ldsm_x4_t(bv, V_s + (size_t)(kb + (lane & 7) + ((lane >> 3) & 1) * 8) * KSTR + p * 16 + (lane >> 4) * 8);
            mma_bf16(O[2 * p], ph, bv[0], bv[1]); mma_bf16(O[2 * p + 1], ph, bv[2], bv[3]);
            mma_bf16(O[2 * p], pl, bv[0], bv[1]); mma_bf16(O[2 * p + 1], pl, bv[2], bv[3]);
        }
    }
    // ---- send this warp's partial: the DS dimensions rank r finishes go to rank r, (max, sum) to every rank
    if (live) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
            l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
        }
        const int src = crank * AT_WARPS + warp;
        const uint32_t acc_a = smem_u32(rx_acc) + (uint32_t)src * GT * DS * 4, ml_a = smem_u32(rx_ml) + (uint32_t)src * GT * 2 * 4;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int d = nt * 8 + 2 * t4;
            const uint32_t dest = (uint32_t)(d / DS), off = (uint32_t)(d % DS) * 4;
            if (g8 < GT) dsmem_st_v2(dsmem_addr(acc_a + (uint32_t)(g8 * DS) * 4 + off, dest), O[nt][0], O[nt][1]);
            if (g8 + 8 < GT) dsmem_st_v2(dsmem_addr(acc_a + (uint32_t)((g8 + 8) * DS) * 4 + off, dest), O[nt][2], O[nt][3]);
        }
        if (t4 == 0) {
#pragma unroll
            for (int dest = 0; dest < AT_CL; ++dest) {
                if (g8 < GT) dsmem_st_v2(dsmem_addr(ml_a + (uint32_t)g8 * 8, (uint32_t)dest), m_run[0], l_run[0]);
                if (g8 + 8 < GT) dsmem_st_v2(dsmem_addr(ml_a + (uint32_t)(g8 + 8) * 8, (uint32_t)dest), m_run[1], l_run[1]);
            }
        }
    }
    cluster_arrive(); cluster_wait();
    // ---- merge the partials of all warps of all live ranks for this rank's output dimensions, in source order
    const int nsrc = min(AT_CL, nsplit) * AT_WARPS;
    float *o_base = a.o + (size_t)rowbase * (a.qh * HD);
    constexpr int DV = DS / 4;
    // an output = (query row, four dimensions); a group of LPO lanes (a power of two, as many as the block affords)
    // shares the sources of one output and folds its partial results with shuffles - the order is fixed by the lane
    // numbers, so the result does not depend on timing
    const int nout = GT * DV;
    int lsh = 0;
    while (lsh < 5 && (nout << (lsh + 1)) <= AT_THREADS) ++lsh;
    const int LPO = 1 << lsh, sub = tid & (LPO - 1);
#pragma unroll 1
    for (int o0 = 0; o0 < nout; o0 += AT_THREADS >> lsh) {
        const int oi = o0 + (tid >> lsh);
        const bool valid = oi < nout;
        const int oc = valid ? oi : 0;
        const int qi = oc / DV, dd = (oc - qi * DV) * 4, d = crank * DS + dd;
        float M = -INFINITY;
#pragma unroll 4
        for (int sidx = sub; sidx < nsrc; sidx += LPO) M = fmaxf(M, rx_ml[((size_t)sidx * GT + qi) * 2]);
#pragma unroll 1
        for (int w = LPO >> 1; w >= 1; w >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, w));
        float den = 0.f;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int sidx = sub; sidx < nsrc; sidx += LPO) {
            const float2 mlv = *reinterpret_cast<const float2 *>(rx_ml + ((size_t)sidx * GT + qi) * 2);
            const float4 v = *reinterpret_cast<const float4 *>(rx_acc + ((size_t)sidx * GT + qi) * DS + dd);
            const float w = mlv.x == -INFINITY ? 0.f : __expf(mlv.x - M);
            den = fmaf(w, mlv.y, den);
            sum.x = fmaf(w, v.x, sum.x); sum.y = fmaf(w, v.y, sum.y); sum.z = fmaf(w, v.z, sum.z); sum.w = fmaf(w, v.w, sum.w);
        }
#pragma unroll 1
        for (int w = LPO >> 1; w >= 1; w >>= 1) {
            den += __shfl_xor_sync(0xffffffffu, den, w);
            sum.x += __shfl_xor_sync(0xffffffffu, sum.x, w); sum.y += __shfl_xor_sync(0xffffffffu, sum.y, w);
            sum.z += __shfl_xor_sync(0xffffffffu, sum.z, w); sum.w += __shfl_xor_sync(0xffffffffu, sum.w, w);
        }
        if (valid && sub == 0) {
            const int gq = (int)((qi * tinv) >> 16), i = qi - gq * T;
            const float inv = 1.0f / den;
            *reinterpret_cast<float4 *>(o_base + (size_t)i * (a.qh * HD) + (kh * G + gq) * HD + d) =
                make_float4(sum.x * inv, sum.y * inv, sum.z * inv, sum.w * inv);
        }
    }
}


// ------------------------------------------------------------------------------------------------
// Long caches (the KV read is the step's largest byte stream): the streaming form.  One CTA of eight warps owns a
// range of `tiles` tiles of 128 cached keys and walks it with two tile buffers: while the warps work on tile t, the
// copies of tile t+1 (K and V, 64 KB) are in flight - one block-wide barrier per tile and nothing else.  The work on a
// tile is warp-local, as in the latency-lean form: warp w takes keys [16 w, 16 w + 16) of the tile, computes their
// scores for all query rows on the tensor cores, keeps the probabilities in registers, folds them into its own running
// (max, sum) and accumulates its own partial output over the whole head dimension.  After the last tile the eight warp
// partials are merged through shared memory (over the tile buffers); a range that is the whole cache writes the
// result, otherwise the CTA publishes its partial and the CTA of the sequence and KV head that arrives last (ticket
// counter, no spinning) merges the ranges in order, so the result does not depend on timing.  No clusters: every SM
// takes the next CTA as soon as it is free.
constexpr int A2_THREADS = 256, A2_WARPS = 8, A2_CK = 128, A2_NBUF = 3;

// Tile buffers hold 128 keys x HD bf16 without padding; the 16-byte chunk c of row r sits at chunk position
// c ^ (r & 7), which keeps the eight rows of an ldmatrix 8x8 block on different banks.  Three K and three V buffers:
// two tiles (128 KB at HD = 128) are in flight while the warps work on a third.
struct Attn2Layout { int kstr; size_t tile_bytes, tile_off, q_off, new_off, rope_off, ml_off, total; };
__host__ __device__ inline Attn2Layout attn2_layout(int hd, int mt) {
    Attn2Layout L;
    L.kstr = hd + 8;                       // padded rows of the query and new-row buffers
    L.tile_bytes = (size_t)A2_CK * hd * 2;
    size_t o = 0;                          // offsets from the first 1024-byte boundary of the dynamic shared memory
    L.tile_off = o; o += 2 * A2_NBUF * L.tile_bytes;               // K0 V0 K1 V1 K2 V2; later the warp partials
    L.q_off = o; o += (size_t)2 * mt * 16 * L.kstr * 2;            // bf16 head | remainder
    L.new_off = o; o += (size_t)2 * 16 * L.kstr * 2;               // the new K | V rows as they are cached: a 16-key group of their own
    L.rope_off = o; o += (size_t)HS_MAX_T * (hd / 2) * 8;
    L.ml_off = o; o += (size_t)(A2_WARPS + 1) * mt * 16 * 2 * 4;   // per warp (max, sum) per row, then the merged pair
    L.total = (o + 127) / 128 * 128 + 1024;
    return L;
}
// a tile of cached K or V rows: a long cache is read once per pass, so the copy is marked evict-first in L2
__device__ __forceinline__ void tma_tile_2d(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
                 :: "r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(pol) : "memory");
}

// PK: the last 16-row query tile is "packed" - it holds at most 8 query rows, their bf16 heads in its rows 0-7 and
// their bf16 remainders in rows 8-15.  One MMA then yields both partial products of a row in the SAME thread (the
// accumulator registers of rows g and g + 8), for the scores and again for P V (probability heads feed rows 0-7 of the
// operand, remainders rows 8-15), so that tile costs half the tensor instructions of a full one.  It serves 1..8 query
// rows (MT = 1) and 17..24 (MT = 2: 20 rows at four query heads per KV head and k = 4).
template <int HD, int MT, bool PK>
__global__ void __launch_bounds__(A2_THREADS, 1) attn2_kernel(const __grid_constant__ AttnArgs a) {
    extern __shared__ __align__(1024) unsigned char smraw[];
    constexpr int CK = A2_CK, GTB = MT * 16, NT = HD / 8, RB = HD * 2;       // RB: bytes of a tile row
    constexpr int PB = (MT - 1) * 16;                                        // first row of the packed tile
    const int split = blockIdx.x, kh = blockIdx.y, lb = blockIdx.z, b = a.b0 + lb;
    const int G = a.qh / a.kvh, T = a.T, GT = G * T;
    const Attn2Layout L = attn2_layout(HD, MT);
    const int KSTR = L.kstr;
    unsigned char *sm = smraw + ((1024u - (smem_u32(smraw) & 1023u)) & 1023u);      // swizzled tiles need 1024-byte alignment
    unsigned char *tile_s = sm + L.tile_off;
    auto Kbuf = [&](int i) { return tile_s + (size_t)(2 * i) * L.tile_bytes; };
    auto Vbuf = [&](int i) { return tile_s + (size_t)(2 * i + 1) * L.tile_bytes; };
    __nv_bfloat16 *Qh_s = reinterpret_cast<__nv_bfloat16 *>(sm + L.q_off);        // [GTB][KSTR]
    __nv_bfloat16 *Ql_s = Qh_s + (size_t)GTB * KSTR;
    __nv_bfloat16 *Kn_s = reinterpret_cast<__nv_bfloat16 *>(sm + L.new_off);      // [16][KSTR]
    __nv_bfloat16 *Vn_s = Kn_s + (size_t)16 * KSTR;
    float2 *rope_s = reinterpret_cast<float2 *>(sm + L.rope_off);
    float *wml_s = reinterpret_cast<float *>(sm + L.ml_off);                      // [A2_WARPS + 1][GTB][2]
    __shared__ int ticket_s;
    __shared__ __align__(8) uint64_t tile_bar[A2_NBUF];                              // one per tile buffer pair: bytes of K and V landed
    __shared__ int tile_done[A2_NBUF];                                               // warps that have finished with the pair's current tile

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t tinv = (65536u + T - 1) / T;
    pdl_trigger();

    // ---- before the wait: kv_len, the first two tiles, the RoPE rows
    const int len = __ldcg(a.kv_len + b) + a.len_off;
    const int SPAN = CK * a.tiles;
    const int nsplit = max(1, (len + SPAN - 1) / SPAN);
    if (split >= nsplit) return;                   // beyond the cache
    if (len < 0 || len + T > a.cap) {
        if (tid == 0 && split == 0 && kh == 0) atomicCAS(a.status, 0, len < 0 ? (int)HS_ERR_DEVICE : (int)HS_ERR_CAPACITY);
        return;
    }
    const bool last = split == nsplit - 1;
    const int c0 = split * SPAN, rc = max(0, min(len, c0 + SPAN) - c0);
    const int ntile = (rc + CK - 1) / CK;
    const int nitem = ntile + (last ? 1 : 0);      // the range that ends the cache also takes the new rows, as one more item
    __nv_bfloat16 *Kb = a.Kc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    __nv_bfloat16 *Vb = a.Vc + ((size_t)b * a.kvh + kh) * a.cap * HD;
    // Cached rows of tile t into buffer pair t % 3: tensor copies of 64 columns x 128 rows (the two halves of a 128-wide
    // head dimension land 16 KB apart), issued by one thread, completion counted in bytes on the pair's barrier.  A tile
    // is fetched whole: rows beyond the cache length hold earlier contents or belong to the next head - they are masked
    // (K) or cleared (V) below; rows beyond the tensor read as zero.
    constexpr int HALVES = HD / 64, HS_ = CK * 128;      // HS_: bytes between the halves of a tile
    const int row00 = (b * a.kvh + kh) * a.cap + c0;
    auto fetch = [&](int t) {              // called by ONE thread
        if (t >= ntile) return;
        uint64_t *bar = &tile_bar[t % A2_NBUF];
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the buffer was last touched by ordinary loads / stores
        mbar_expect_tx(bar, 2u * CK * RB);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) {
            tma_tile_2d(Kbuf(t % A2_NBUF) + hf * HS_, &a.kmap, hf * 64, row00 + t * CK, bar);
            tma_tile_2d(Vbuf(t % A2_NBUF) + hf * HS_, &a.vmap, hf * 64, row00 + t * CK, bar);
        }
    };
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < A2_NBUF; ++i) { mbar_init(&tile_bar[i], 1); tile_done[i] = 0; }
        mbar_fence_init();
    }
    if (tid == 0) { fetch(0); fetch(1); fetch(2); }
#pragma unroll 1
    for (int idx = tid; idx < T * (HD / 2); idx += A2_THREADS) {
        const int i = idx / (HD / 2), e = idx - i * (HD / 2);
        rope_s[idx] = a.rope[(size_t)(len + i) * (HD / 2) + e];
    }
#pragma unroll 1
    for (int idx = tid; idx < (GTB - GT) * (HD / 8); idx += A2_THREADS) {      // query rows that do not exist are zero
        const int r = GT + idx / (HD / 8), c = idx % (HD / 8);
        *reinterpret_cast<uint4 *>(Qh_s + (size_t)r * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4 *>(Ql_s + (size_t)r * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
    }
#pragma unroll 1
    for (int idx = tid; idx < 16 * (HD / 8); idx += A2_THREADS) {              // finite V rows behind the new ones
        const int r = idx / (HD / 8), c = idx % (HD / 8);
        *reinterpret_cast<uint4 *>(Vn_s + (size_t)r * KSTR + 8 * c) = make_uint4(0, 0, 0, 0);
    }
    pdl_wait();
    __syncthreads();                        // rope_s complete, Vn_s cleared

    // ---- queries (RoPE, scale, bf16 head + remainder) and, in the last range, the new K / V rows
    const int rowbase = lb * T;
    const float scale = rsqrtf((float)HD);
    {
        constexpr int HP = HD / 2, NH = A2_THREADS / HP;
        const int e = tid % HP, part = tid / HP;
#pragma unroll 1
        for (int q0 = part; q0 < GT; q0 += 4 * NH) {
            float x0[4], x1[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int qi = q0 + u * NH;
                x0[u] = x1[u] = 0.f;
                if (qi < GT) {
                    const int gq = (int)((qi * tinv) >> 16);
                    const float *src = a.zx + (size_t)(rowbase + qi - gq * T) * a.in_ld + a.q_off + (kh * G + gq) * HD;
                    x0[u] = __ldcg(src + e); x1[u] = __ldcg(src + e + HP);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int qi = q0 + u * NH;
                if (qi < GT) {
                    const float2 cs = rope_s[(qi - (int)((qi * tinv) >> 16) * T) * HP + e];
                    __nv_bfloat16 h, l;
                    // the remainder of a row of the packed tile lives eight rows further down the same array
                    __nv_bfloat16 *lo_row = (PK && qi >= PB) ? Qh_s + (size_t)(qi + 8) * KSTR : Ql_s + (size_t)qi * KSTR;
                    split_bf16((x0[u] * cs.x - x1[u] * cs.y) * scale, h, l);
                    Qh_s[qi * KSTR + e] = h; lo_row[e] = l;
                    split_bf16((x1[u] * cs.x + x0[u] * cs.y) * scale, h, l);
                    Qh_s[qi * KSTR + e + HP] = h; lo_row[e + HP] = l;
                }
            }
        }
    }
    if (last) {
#pragma unroll 1
        for (int idx = tid; idx < T * (HD / 2); idx += A2_THREADS) {
            const int i = idx / (HD / 2), e = idx - i * (HD / 2);
            const float *row = a.zx + (size_t)(rowbase + i) * a.in_ld;
            const float2 cs = rope_s[idx];
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
    __syncthreads();                        // queries and new rows in place

    const int g8 = lane >> 2, t4 = lane & 3;
    float O[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { O[mt][nt][0] = O[mt][nt][1] = O[mt][nt][2] = O[mt][nt][3] = 0.f; }
    float m_run[MT][2], l_run[MT][2];
    int ti[MT][2];                          // position index of each of this lane's rows among the T new ones
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            m_run[mt][r] = -INFINITY; l_run[mt][r] = 0.f;
            const int row = mt * 16 + g8 + 8 * r;
            ti[mt][r] = row - (int)((row * tinv) >> 16) * T;
        }

    // An item is a tile of cached keys (a buffer of the ring, swizzled rows of RB bytes) or, last, the new rows (their own
    // padded buffer): the same code serves both, told apart by base address, row pitch and swizzle mask.
#pragma unroll 1
    for (int t = 0; t < nitem; ++t) {
        const bool newrows = t >= ntile;
        const int nkeys = newrows ? T : min(CK, rc - t * CK);
        const int nkp = (nkeys + 15) & ~15;
        if (!newrows) {
            // Tile t has landed (tiles t + 1 and t + 2 may be in flight); a wait that runs out is reported and the pass goes
            // on.  There is no block-wide barrier per tile: a warp works on its 16 keys as soon as the tile is there and
            // hands the buffers back when it is done (below), so the warps drift apart and fill each other's stalls.
            if (!mbar_wait(&tile_bar[t % A2_NBUF], (uint32_t)(t / A2_NBUF) & 1u) && lane == 0) atomicCAS(a.status, 0, (int)HS_ERR_TIMEOUT);
            if (nkp != nkeys && warp * 16 <= nkeys && nkeys < warp * 16 + 16) {
                // a ragged tile (only the last can be): finite V rows for the padding keys of the group that holds them
                unsigned char *vd = Vbuf(t % A2_NBUF);
#pragma unroll 1
                for (int idx = lane; idx < (nkp - nkeys) * (HD / 8); idx += 32) {
                    const int c = idx % (HD / 8);
                    *reinterpret_cast<uint4 *>(vd + (c >> 3) * HS_ + (size_t)(nkeys + idx / (HD / 8)) * 128 + ((c & 7) << 4)) = make_uint4(0, 0, 0, 0);
                }
                __syncwarp();
            }
        }
        const unsigned char *K_s = newrows ? reinterpret_cast<const unsigned char *>(Kn_s) : Kbuf(t % A2_NBUF);
        const unsigned char *V_s = newrows ? reinterpret_cast<const unsigned char *>(Vn_s) : Vbuf(t % A2_NBUF);
        // a tile: rows of 128 bytes per half, 16-byte chunks XOR-swizzled with the row; the new rows: padded rows, no swizzle
        const int pitch = newrows ? KSTR * 2 : 128, swz = newrows ? 0 : 7, hstr = newrows ? 128 : HS_;
        // 16 keys per warp; the new rows are one group, given to the warp that a ragged last tile leaves idle most often
#pragma unroll 1
        for (int kb = (newrows ? (warp == A2_WARPS - 1 ? 0 : nkp) : warp * 16); kb < nkp; kb += A2_WARPS * 16) {
            // ---- scores of this warp's 16 keys for all query rows (two accumulator sets: head and remainder products)
            float S[MT][2][4];
            {
                float Sp[2][MT][2][4];
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int nt = 0; nt < 2; ++nt) { Sp[c][mt][nt][0] = Sp[c][mt][nt][1] = Sp[c][mt][nt][2] = Sp[c][mt][nt][3] = 0.f; }
                const int krow = kb + (lane & 7) + (lane >> 4) * 8;
                const unsigned char *krp = K_s + (size_t)krow * pitch;
                const int ksw = krow & swz, kc0 = (lane >> 3) & 1;
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    uint32_t bk[4];
                    ldsm_x4(bk, krp + ((ks * 2 + kc0) >> 3) * hstr + (((((ks * 2 + kc0) & 7)) ^ ksw) << 4));
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        uint32_t ah[4], al[4];
                        const size_t qo = (size_t)(mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * KSTR + ks * 16 + (lane >> 4) * 8;
                        ldsm_x4(ah, Qh_s + qo);
                        mma_bf16(Sp[0][mt][0], ah, bk[0], bk[1]); mma_bf16(Sp[0][mt][1], ah, bk[2], bk[3]);
                        if (!(PK && mt == MT - 1)) {
                            ldsm_x4(al, Ql_s + qo);
                            mma_bf16(Sp[1][mt][0], al, bk[0], bk[1]); mma_bf16(Sp[1][mt][1], al, bk[2], bk[3]);
                        }
                    }
                }
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) S[mt][nt][e] = Sp[0][mt][nt][e] + Sp[1][mt][nt][e];
                if (PK)                      // packed tile: head product in the registers of row g, remainder product in those of row g + 8
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) { S[MT - 1][nt][0] += S[MT - 1][nt][2]; S[MT - 1][nt][1] += S[MT - 1][nt][3]; }
            }
            // ---- masks, running softmax, probabilities as operand fragments
            const bool edge = newrows || kb + 16 > nkeys;
            uint32_t ph[MT][4], pl[MT][4];
            float corr_all[MT][2];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                float mx[2] = {-INFINITY, -INFINITY};
                if (edge) {                 // only a ragged last group and the new rows have anything to mask
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int key = kb + nt * 8 + 2 * t4 + (e & 1);
                            if (key >= nkeys || (newrows && key > ti[mt][e >> 1])) S[mt][nt][e] = -INFINITY;
                        }
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) mx[e >> 1] = fmaxf(mx[e >> 1], S[mt][nt][e]);
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const bool packed = PK && mt == MT - 1;
                    if (packed && r == 1) { corr_all[mt][1] = corr_all[mt][0]; continue; }   // rows 8-15 carry remainders, not rows
                    mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                    mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                    const float mnew = fmaxf(m_run[mt][r], mx[r]);
                    const float muse = mnew == -INFINITY ? 0.f : mnew;
                    const float corr = __expf(m_run[mt][r] - muse);
                    corr_all[mt][r] = corr;
                    m_run[mt][r] = mnew;
                    float sum = 0.f;
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt) {
                        const float p0 = __expf(S[mt][nt][2 * r] - muse), p1 = __expf(S[mt][nt][2 * r + 1] - muse);
                        sum += p0 + p1;
                        // two probabilities at a time: bf16 heads packed by one conversion, remainders from the exact differences
                        const uint32_t hh = pack_bf16x2(p0, p1);
                        const uint32_t ll = pack_bf16x2(p0 - __uint_as_float(hh << 16), p1 - __uint_as_float(hh & 0xffff0000u));
                        ph[mt][r + 2 * nt] = hh;
                        if (packed) ph[mt][1 + 2 * nt] = ll;     // operand rows 8-15 of the packed tile
                        else pl[mt][r + 2 * nt] = ll;
                    }
                    l_run[mt][r] = fmaf(l_run[mt][r], corr, sum);
                }
            }
            // the accumulators are rescaled only when some row's running maximum moved (rare after the first tiles)
            bool moved = false;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) moved = moved || corr_all[mt][0] != 1.f || corr_all[mt][1] != 1.f;
            if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        O[mt][nt][0] *= corr_all[mt][0]; O[mt][nt][1] *= corr_all[mt][0];
                        O[mt][nt][2] *= corr_all[mt][1]; O[mt][nt][3] *= corr_all[mt][1];
                    }
            }
            // ---- partial output += P V over the whole head dimension
            const int vrow = kb + (lane & 7) + ((lane >> 3) & 1) * 8;
            const unsigned char *vrp = V_s + (size_t)vrow * pitch;
            const int vsw = vrow & swz, vc0 = lane >> 4;
#pragma unroll
            for (int p = 0; p < NT / 2; ++p) {
                uint32_t bv[4];
                ldsm_x4_t(bv, vrp + ((p * 2 + vc0) >> 3) * hstr + ((((p * 2 + vc0) & 7) ^ vsw) << 4));
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    mma_bf16(O[mt][2 * p], ph[mt], bv[0], bv[1]); mma_bf16(O[mt][2 * p + 1], ph[mt], bv[2], bv[3]);
                    if (!(PK && mt == MT - 1)) {
                        mma_bf16(O[mt][2 * p], pl[mt], bv[0], bv[1]); mma_bf16(O[mt][2 * p + 1], pl[mt], bv[2], bv[3]);
                    }
                }
            }
        }
        if (!newrows) {
            // this warp is done with tile t: the last of the eight to say so refills the buffer pair with tile t + 3
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                if (atomicAdd(&tile_done[t % A2_NBUF], 1) == A2_WARPS - 1) { tile_done[t % A2_NBUF] = 0; fetch(t + A2_NBUF); }
            }
        }
    }
    __syncthreads();                        // everybody is done with the tile buffers (every requested tile was waited for)

    // ---- merge the eight warp partials through shared memory (the tile buffers are free now)
    float *wo_s = reinterpret_cast<float *>(sm + L.tile_off);            // [A2_WARPS][GTB][HD]
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const bool packed = PK && mt == MT - 1;
            if (packed && r == 1) continue;
            if (packed)                       // head and remainder halves of the packed tile's outputs
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) { O[mt][nt][0] += O[mt][nt][2]; O[mt][nt][1] += O[mt][nt][3]; }
            float l = l_run[mt][r];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int row = mt * 16 + g8 + 8 * r;
            if (t4 == 0) { wml_s[((size_t)warp * GTB + row) * 2] = m_run[mt][r]; wml_s[((size_t)warp * GTB + row) * 2 + 1] = l; }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                *reinterpret_cast<float2 *>(wo_s + ((size_t)warp * GTB + row) * HD + nt * 8 + 2 * t4) = make_float2(O[mt][nt][2 * r], O[mt][nt][2 * r + 1]);
        }
    __syncthreads();
    float *o_base = a.o + (size_t)rowbase * (a.qh * HD);
    const size_t pslot = ((size_t)b * a.kvh + kh) * a.nch + split;
    float *mrg_s = wml_s + (size_t)A2_WARPS * GTB * 2;                       // [GTB][2] merged (M, den)
    constexpr int DV4 = HD / 4;
#pragma unroll 1
    for (int idx = tid; idx < GT * DV4; idx += A2_THREADS) {
        const int qi = idx / DV4, d = (idx - qi * DV4) * 4;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < A2_WARPS; ++w) M = fmaxf(M, wml_s[((size_t)w * GTB + qi) * 2]);
        float den = 0.f;
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < A2_WARPS; ++w) {
            const float mw = wml_s[((size_t)w * GTB + qi) * 2];
            const float wt = mw == -INFINITY ? 0.f : __expf(mw - M);
            den = fmaf(wt, wml_s[((size_t)w * GTB + qi) * 2 + 1], den);
            const float4 v = *reinterpret_cast<const float4 *>(wo_s + ((size_t)w * GTB + qi) * HD + d);
            sum.x = fmaf(wt, v.x, sum.x); sum.y = fmaf(wt, v.y, sum.y); sum.z = fmaf(wt, v.z, sum.z); sum.w = fmaf(wt, v.w, sum.w);
        }
        if (nsplit == 1) {
            const int gq = (int)((qi * tinv) >> 16), i = qi - gq * T;
            const float inv = 1.0f / den;
            *reinterpret_cast<float4 *>(o_base + (size_t)i * (a.qh * HD) + (kh * G + gq) * HD + d) =
                make_float4(sum.x * inv, sum.y * inv, sum.z * inv, sum.w * inv);
        } else {
            *reinterpret_cast<float4 *>(a.part_acc + pslot * HS_MAX_GT * HD + (size_t)qi * HD + d) = sum;
            if (d == 0) { mrg_s[2 * qi] = M; mrg_s[2 * qi + 1] = den; }
        }
    }
    if (nsplit == 1) return;
    __syncthreads();
    if (tid < 2 * GT) a.part_ml[pslot * HS_MAX_GT * 2 + tid] = mrg_s[tid];
    // ---- several ranges: the CTA that arrives last merges their partials in order
    __threadfence();
    __syncthreads();
    if (tid == 0) ticket_s = atomicAdd(a.counters + b * a.kvh + kh, 1);
    __syncthreads();
    if (ticket_s != nsplit - 1) return;
    __threadfence();
    if (tid == 0) a.counters[b * a.kvh + kh] = 0;          // ready for the next launch
    const size_t pbase = ((size_t)b * a.kvh + kh) * a.nch;
    const float *pa0 = a.part_acc + pbase * HS_MAX_GT * HD;
    const float *pm0 = a.part_ml + pbase * HS_MAX_GT * 2;
    for (int qi = warp; qi < GT; qi += A2_WARPS) {
        float M = -INFINITY;
        for (int c = lane; c < nsplit; c += 32) M = fmaxf(M, __ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
        M = warp_max(M);
        float den = 0.f;
        for (int c = lane; c < nsplit; c += 32) {
            const float2 mlv = __ldcg(reinterpret_cast<const float2 *>(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2));
            den = fmaf(__expf(mlv.x - M), mlv.y, den);
        }
        den = warp_sum(den);
        if (lane == 0) { mrg_s[2 * qi] = M; mrg_s[2 * qi + 1] = den; }
    }
    __syncthreads();
#pragma unroll 1
    for (int idx = tid; idx < GT * DV4; idx += A2_THREADS) {
        const int qi = idx / DV4, d = (idx - qi * DV4) * 4;
        const float M = mrg_s[2 * qi];
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int c = 0; c < nsplit; ++c) {
            const float wt = __expf(__ldcg(pm0 + ((size_t)c * HS_MAX_GT + qi) * 2) - M);
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(pa0 + ((size_t)c * HS_MAX_GT + qi) * HD + d));
            sum.x = fmaf(wt, v.x, sum.x); sum.y = fmaf(wt, v.y, sum.y); sum.z = fmaf(wt, v.z, sum.z); sum.w = fmaf(wt, v.w, sum.w);
        }
        const int gq = (int)((qi * tinv) >> 16), i = qi - gq * T;
        const float inv = 1.0f / mrg_s[2 * qi + 1];
        *reinterpret_cast<float4 *>(o_base + (size_t)i * (a.qh * HD) + (kh * G + gq) * HD + d) =
            make_float4(sum.x * inv, sum.y * inv, sum.z * inv, sum.w * inv);
    }
}

template <int HD, int MT, bool PK>
cudaError_t launch_attn2_t(const AttnArgs &a, cudaStream_t s) {
    static bool configured = false;
    const size_t smem = attn2_layout(HD, MT).total;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(attn2_kernel<HD, MT, PK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn2_kernel<HD, MT, PK>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_pdl(attn2_kernel<HD, MT, PK>, dim3(a.nch, a.kvh, a.nb), dim3(A2_THREADS), smem, s, a);
}

template <int HD, int MT>
__global__ void __launch_bounds__(AT_THREADS) attn_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char smraw[];
    attn_body<HD, MT>(a, blockIdx.x, blockIdx.y, blockIdx.z, smraw);
}

// Verify pass of a parallel hybrid block: the Mamba-2 mixer and the attention read the same in-projection
// output and feed the same out-projection, so they run as ONE launch - the first `attn_ctas` blocks (whole
// clusters) are attention CTAs, the rest mixer CTAs - and the dependent-launch chain is one kernel shorter.
struct FusedGeo { int attn_nx, attn_ctas, ssm_nx, ssm_ctas; };

template <int HD>
__global__ void __launch_bounds__(AT_THREADS) attn_small_kernel(const AttnArgs a) {
    extern __shared__ __align__(128) unsigned char smraw[];
    attn_small_body<HD>(a, blockIdx.x, blockIdx.y, blockIdx.z, smraw);
}

// MT = 0 selects the latency-lean attention body (few query rows, cache within one cluster)
template <int EPL, int HD, int MT, int TMAX>
__global__ void __launch_bounds__(AT_THREADS) ssm_attn_kernel(const SsmArgs sa, const AttnArgs aa, const FusedGeo g) {
    extern __shared__ __align__(128) unsigned char smraw[];
    const int id = blockIdx.x;
    if (id < g.attn_ctas) {
        const int split = id % g.attn_nx, t = id / g.attn_nx;
        if (MT == 0) attn_small_body<HD>(aa, split, t % aa.kvh, t / aa.kvh, smraw);
        else attn_body<HD, MT == 0 ? 1 : MT>(aa, split, t % aa.kvh, t / aa.kvh, smraw);
    } else if (id - g.attn_ctas < g.ssm_ctas) {
        const int j = id - g.attn_ctas, bx = j % g.ssm_nx, t = j / g.ssm_nx;
        ssm_body<EPL, 16, TMAX>(sa, bx, t % sa.H, t / sa.H);
    }
}

template <int HD, int MT>
cudaError_t launch_t(const AttnArgs &a, cudaStream_t s) {
    dim3 grid((a.nch + AT_CL - 1) / AT_CL * AT_CL, a.kvh, a.nb);
    const size_t smem = attn_layout(HD, a.chunk, (a.qh / a.kvh) * a.T).total;
    return launch_pdl_cluster(attn_kernel<HD, MT>, grid, dim3(AT_THREADS), smem, s, AT_CL, a);
}

template <int HD>
cudaError_t launch_small_t(const AttnArgs &a, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(attn_small_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_small_layout(HD, AT_SMALL_MAXCHUNK, 16).total);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_small_kernel<HD>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const size_t smem = attn_small_layout(HD, a.chunk, (a.qh / a.kvh) * a.T).total;
    return launch_pdl_cluster(attn_small_kernel<HD>, dim3(AT_CL, a.kvh, a.nb), dim3(AT_THREADS), smem, s, AT_CL, a);
}

template <int EPL, int HD, int MT, int TMAX>
cudaError_t launch_fused_t(const SsmArgs &sa, const AttnArgs &a, cudaStream_t s) {
    FusedGeo g;
    g.attn_nx = MT == 0 ? AT_CL : (a.nch + AT_CL - 1) / AT_CL * AT_CL;
    g.attn_ctas = g.attn_nx * a.kvh * a.nb;
    g.ssm_nx = sa.P / 16;
    g.ssm_ctas = g.ssm_nx * sa.H * sa.nb;
    const int total = (g.attn_ctas + g.ssm_ctas + AT_CL - 1) / AT_CL * AT_CL;
    const size_t smem = MT == 0 ? attn_small_layout(HD, a.chunk, (a.qh / a.kvh) * a.T).total : attn_layout(HD, a.chunk, (a.qh / a.kvh) * a.T).total;
    static bool configured = false;
    if (!configured) {
        const size_t most = MT == 0 ? attn_small_layout(HD, AT_SMALL_MAXCHUNK, 16).total : attn_layout(HD, 128, MT * 16).total;
        cudaError_t e = cudaFuncSetAttribute(ssm_attn_kernel<EPL, HD, MT, TMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(ssm_attn_kernel<EPL, HD, MT, TMAX>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    return launch_pdl_cluster(ssm_attn_kernel<EPL, HD, MT, TMAX>, dim3(total), dim3(AT_THREADS), smem, s, AT_CL, sa, a, g);
}

template <int HD, int MT>
cudaError_t configure_t() {
    cudaError_t e = cudaFuncSetAttribute(attn_kernel<HD, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_layout(HD, 128, MT * 16).total);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_kernel<HD, MT>, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    return e;
}

}  // namespace

cudaError_t configure_attn() {
    cudaError_t e = configure_t<128, 1>();
    if (e == cudaSuccess) e = configure_t<128, 2>();
    if (e == cudaSuccess) e = configure_t<128, 3>();
    if (e == cudaSuccess) e = configure_t<64, 1>();
    if (e == cudaSuccess) e = configure_t<64, 2>();
    if (e == cudaSuccess) e = configure_t<64, 3>();
    return e;
}

cudaError_t launch_attn(const AttnArgs &a, cudaStream_t s) {
    const int GT = (a.qh / a.kvh) * a.T;
    if (a.small) {
        if (GT > 16 || a.chunk < 16 || a.chunk > AT_SMALL_MAXCHUNK || (a.chunk & 15)) return cudaErrorInvalidValue;
        return a.hd == 128 ? launch_small_t<128>(a, s) : a.hd == 64 ? launch_small_t<64>(a, s) : cudaErrorInvalidValue;
    }
    if (a.stream) {          // the streaming form: 128-key tiles, a.tiles of them per CTA, at most 32 query rows
        if (GT > 32 || a.chunk != A2_CK || a.tiles < 1) return cudaErrorInvalidValue;
        // at most 8 rows in the last 16-row tile: the packed form of that tile (half its tensor instructions)
#define A2(hd_) if (a.hd == hd_) return GT <= 8 ? launch_attn2_t<hd_, 1, true>(a, s) : GT <= 16 ? launch_attn2_t<hd_, 1, false>(a, s) \
                                      : GT <= 24 ? launch_attn2_t<hd_, 2, true>(a, s) : launch_attn2_t<hd_, 2, false>(a, s)
        A2(128); A2(64);
#undef A2
        return cudaErrorInvalidValue;
    }
    if (GT > HS_MAX_GT || a.chunk < 16 || a.chunk > 128 || (a.chunk & 15) || a.tiles < 1) return cudaErrorInvalidValue;
    const int mt = (GT + 15) / 16;
#define CASE(hd_, m_) if (a.hd == hd_ && mt == m_) return launch_t<hd_, m_>(a, s)
    CASE(128, 1); CASE(128, 2); CASE(128, 3); CASE(64, 1); CASE(64, 2); CASE(64, 3);
#undef CASE
    return cudaErrorInvalidValue;
}

// Fused launch for a parallel block of the verify pass; `fused` reports whether it applies (mixer blocks of
// 16 state rows, 128 threads in both roles) - otherwise nothing is launched and the caller issues the two
// kernels one after the other.
cudaError_t launch_ssm_attn(const SsmArgs &sa, const AttnArgs &a, cudaStream_t s, bool *fused) {
    const int GT = (a.qh / a.kvh) * a.T, mt = a.small ? 0 : (GT + 15) / 16;
    *fused = false;
    if (ssm_wide(sa) || GT > HS_MAX_GT || a.tiles < 1 || a.chunk < 16 || a.chunk > 128 || (a.chunk & 15) || sa.P % 16) return cudaSuccess;
    // In the fused launch every mixer block carries the attention's shared-memory allocation.  With a few blocks per SM
    // (batch 1) that costs nothing and saves a kernel on the dependent chain; with many (larger batches) it caps the
    // number of resident mixer blocks and with it the state bandwidth: then the two kernels go out separately.
    if ((int64_t)(sa.P / 16) * sa.H * sa.nb > 4 * 148) return cudaSuccess;
    if (a.small && GT > 16) return cudaErrorInvalidValue;
#define CASE(n_, e_, hd_, m_) if (sa.N == n_ && a.hd == hd_ && mt == m_) { *fused = true; return a.T <= 3 ? launch_fused_t<e_, hd_, m_, 3>(sa, a, s) : launch_fused_t<e_, hd_, m_, HS_MAX_T>(sa, a, s); }
#define CASES(n_, e_) CASE(n_, e_, 128, 0) CASE(n_, e_, 64, 0) CASE(n_, e_, 128, 1) CASE(n_, e_, 128, 2) CASE(n_, e_, 128, 3) CASE(n_, e_, 64, 1) CASE(n_, e_, 64, 2) CASE(n_, e_, 64, 3)
    CASES(64, 2) CASES(128, 4) CASES(256, 8)
#undef CASES
#undef CASE
    return cudaSuccess;
}

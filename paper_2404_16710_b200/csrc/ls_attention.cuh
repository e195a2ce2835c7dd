// Decode / verify attention over the paged bf16 KV cache (one KV cache shared by the draft
// and the verify stage, LayerSkip Sec. 4.3.3), for passes of up to 16 rows.
//
// One thread-block cluster per KV head.  The keys are cut by ABSOLUTE position into spans of
// R chunks of 64 keys; CTA k of the cluster owns span k (keys [64 R k, 64 R (k+1))), streams its
// chunks through a two-stage cp.async ring and keeps a running (max, sum, weighted values) per
// query -- the online-softmax recurrence, chunk after chunk in position order.  The spans'
// results never go through global memory: every CTA leaves (max, sum, values) in its own shared
// memory, the cluster meets at a barrier, and each CTA then combines a slice of the
// (query, dim) outputs by reading all spans through distributed shared memory, in span order.
// No counters, no fences, no second kernel.
//
// R = ceil(ceil(max_seq / 64) / cluster size) is a constant of the model, so what a row's
// result depends on is its position alone: a chunk or a span that lies wholly beyond the row's
// position leaves its running state bit for bit as it was (weights 0, scale factor exp(0)),
// which makes the verify pass of d+1 rows (Sec. 4.3.2) reproduce single-token decoding exactly,
// whatever the pass size and whatever later rows share the launch.
//
// q.k and p.v run on the tensor cores (mma.sync.m16n8k16, fp32 accumulate) at every pass size:
// the queries of the KV head's group (rows x G) are the 16-row operand in tiles of 16,
// zero-padded.  q.k: warp w owns keys 8w..8w+7 of the chunk; a thread's 16-byte pieces of its
// query rows and of its key row are its fragments (the contraction index is permuted alike on
// both sides).  p.v: p is rounded to bf16, warp w owns 16 (HD 128) or 8 (HD 64) output dims,
// V fragments come transposed out of ldmatrix.  Row pitches keep every access pattern free of
// bank conflicts: K and Q rows 64 mod 128 bytes, V rows 16 mod 128 bytes.
#pragma once
#include "ls_kernels.cuh"

namespace ls {

constexpr int kAttnStages = 2;       // K/V chunks in flight per CTA
constexpr int kAttnMaxCluster = 8;   // portable cluster size

// launch shape of the attention kernel for one model: CTAs per cluster, chunks of 64 keys per CTA
struct AttnPlan {
    int csize, span;
};

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr)
{
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float ld_cluster_f(uint32_t addr)
{
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}

// shared memory: stage[2] { Ks [64][HD*2+64 B] | Vs [64][HD*2+16 B] } | Qb bf16 [Qpad][HD*2+64 B]
//                | S f32 [Qpad][72] | Pb bf16 [Qpad][72] | Mrun, Lrun, Alpha f32 [Qpad] each
// (Qpad = Q rounded up to 16); after the last chunk the stage area holds the CTA's
// un-normalised values Om f32 [Qpad][HD] for the other CTAs of the cluster to read.
template <int HD>
__host__ __device__ constexpr size_t attn_stage_bytes()
{
    return (size_t)kAttnChunk * (HD * 2 + 64) + (size_t)kAttnChunk * (HD * 2 + 16);
}
template <int HD>
__host__ __device__ constexpr size_t attn_smem_bytes(int Q)
{
    const size_t qpad = ((size_t)Q + 15) / 16 * 16;
    return kAttnStages * attn_stage_bytes<HD>() + qpad * (HD * 2 + 64) + qpad * kAttnSP * 4 + qpad * kAttnSP * 2 +
           3 * qpad * sizeof(float);
}

// grid (cluster size, Hkv), cluster (cluster size, 1, 1), block 256.  QT: tiles of 16 queries
// the instantiation can hold (Q = G * M <= 16 QT).  span_chunks: R above.
template <int HD, int QT>
__global__ void __launch_bounds__(kAttnThreads)
attn_cluster_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ kpages,
                    const uint16_t* __restrict__ vpages, const int32_t* __restrict__ page_table,
                    int32_t* ctl, int pos_off, int M, int Hq, int Hkv, int page_shift,
                    int max_seq, int span_chunks, uint16_t* __restrict__ out, int gate)
{
    constexpr int C = kAttnChunk, T = kAttnThreads, NST = kAttnStages;
    constexpr int KROW = HD * 2 + 64, VROW = HD * 2 + 16;
    constexpr int SP = kAttnSP, PBROW = kAttnSP * 2;
    constexpr int SEGS = HD * 2 / 16;  // 16-byte segments per row
    constexpr int NTW = HD / 64;       // n8 tiles of output dims per warp: 2 (HD 128) or 1 (HD 64)
    constexpr size_t STAGE = attn_stage_bytes<HD>();
    static_assert(STAGE % 16 == 0, "stages keep 16-byte alignment");
    extern __shared__ __align__(16) unsigned char smem[];
    const int kh = blockIdx.y, tid = threadIdx.x;
    const int rank = (int)cluster_ctarank(), csize = (int)gridDim.x;
    const int warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    const int chunk0 = rank * span_chunks;  // first chunk of this CTA's span
    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(smem);
    const bool one_page = page_shift >= 6;  // a chunk never straddles a page of 64 tokens or more

    // rows p of chunk c with p_lo <= p <= p_hi are copied into stage s; rows p_hi < p <= p_fill are zeroed
    auto stage_rows = [&](int c, int s, int p_lo, int p_hi, int p_fill) {
        const int key0 = c * C;
        const uint32_t ks0 = smem0 + (uint32_t)(s * STAGE), vs0 = ks0 + C * KROW;
        size_t base = 0;
        if (one_page) base = kv_row_offset(page_table, key0, page_shift, Hkv, kh, HD);
#pragma unroll
        for (int it = 0; it < C * SEGS / T; ++it) {
            const int idx = tid + it * T;
            const int r = idx / SEGS, sg = idx % SEGS;
            const int p = key0 + r;
            if (p < p_lo || p > p_fill) continue;
            const bool ok = p <= p_hi;
            const size_t off = (one_page ? base + (size_t)r * HD
                                         : kv_row_offset(page_table, ok ? p : key0, page_shift, Hkv, kh, HD)) +
                               (size_t)sg * 8;
            cp_async16_cg(ks0 + r * KROW + sg * 16, kpages + off, ok ? 16 : 0);
            cp_async16_cg(vs0 + r * VROW + sg * 16, vpages + off, ok ? 16 : 0);
        }
    };

    // Cache rows below the loop's cache length do not change while the loop runs, so their
    // copies start before the producer of q (and of this pass's own k, v rows) has finished.
    // The length is read past L1 and may be an older, smaller one: then fewer rows go early.
    pdl_launch_dependents();
    int c_early = 0;
    if (ctl && !(gate > 0 && gate > __ldcg(ctl + CTL_D_EFF))) c_early = min(__ldcg(ctl + CTL_CACHE_LEN), max_seq);
#pragma unroll
    for (int s = 0; s < NST; ++s)
        if (s < span_chunks && (chunk0 + s) * C < c_early) stage_rows(chunk0 + s, s, 0, c_early - 1, c_early - 1);
    pdl_wait();
    auto drain = [&]() {  // nothing in flight may outlive the CTA's shared memory
        cp_async_commit();
        cp_async_wait<0>();
    };
    // the three ways out below are taken by every CTA of the grid alike (they depend on the
    // control words and the launch arguments only), so no CTA is left waiting at a cluster barrier
    if (pass_idle(ctl, gate)) return drain();
    const int pos0 = (ctl ? ctl[CTL_CACHE_LEN] : 0) + pos_off;
    const int last_pos = pos0 + M - 1;
    const int G = Hq / Hkv, Q = G * M;  // query qi = m * G + g
    const int Qpad = (Q + 15) & ~15;
    if (last_pos >= max_seq || pos0 < 0 || last_pos / (C * span_chunks) >= csize || Qpad > 16 * QT) {
        if (ctl && tid == 0) ctl[CTL_STATUS] = DEV_POS_OVERFLOW;
        return drain();
    }
    if (c_early > pos0) c_early = pos0;  // (cannot happen: the length only grows; rows >= pos0 are this pass's)
    const int n_active = last_pos / (C * span_chunks) + 1;  // spans with a visible key
    // chunks this CTA walks: its span, cut at the last visible key
    const int nc = rank < n_active ? min(span_chunks, last_pos / C + 1 - chunk0) : 0;

    unsigned char* Qb = smem + NST * STAGE;
    float* S = reinterpret_cast<float*>(Qb + (size_t)Qpad * KROW);
    unsigned char* Pb = reinterpret_cast<unsigned char*>(S + (size_t)Qpad * SP);
    float* Mrun = reinterpret_cast<float*>(Pb + (size_t)Qpad * PBROW);
    float* Lrun = Mrun + Qpad;
    float* Alpha = Lrun + Qpad;
    float* Om = reinterpret_cast<float*>(smem);  // [Qpad][HD], over the stages once they are drained

    // the remaining rows of the first chunks (zeros beyond the last visible key), one commit
    // group per chunk slot, empty when the span has no such chunk
#pragma unroll
    for (int s = 0; s < NST; ++s) {
        if (s < nc) stage_rows(chunk0 + s, s, c_early, last_pos, (chunk0 + s) * C + C - 1);
        cp_async_commit();
    }
    if (nc > 0) {
        // the group's queries (bf16, 16-byte pieces) and the running state
        const int nq = Qpad * SEGS;
        for (int idx = tid; idx < nq; idx += T) {
            const int qi = idx / SEGS, sg = idx % SEGS;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (qi < Q) {
                const int m = qi / G, g = qi % G;
                v = *reinterpret_cast<const uint4*>(q + ((size_t)m * Hq + (size_t)kh * G + g) * HD + sg * 8);
            }
            *reinterpret_cast<uint4*>(Qb + qi * KROW + sg * 16) = v;
        }
        for (int qi = tid; qi < Qpad; qi += T) {
            Mrun[qi] = -INFINITY;
            Lrun[qi] = 0.f;
        }
    }

    float acc[QT][NTW][4];
#pragma unroll
    for (int t = 0; t < QT; ++t)
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t][nt][i] = 0.f;

    const float scale = rsqrtf((float)HD);
    const int d0 = NTW * 8 * warp;  // this warp's output dims in p.v
    // ldmatrix: lane L addresses row L%8 of matrix L/8; matrices 0, 1: keys 0-7, 8-15 of the
    // 16-key block at dims d0..d0+7; matrices 2, 3: the same keys at dims d0+8..
    const int mi = lane >> 3, mr = lane & 7;
    const uint32_t vlane_off = (uint32_t)(((mi & 1) * 8 + mr) * VROW + (d0 + ((NTW == 2) ? (mi >> 1) * 8 : 0)) * 2);

    for (int i = 0; i < nc; ++i) {
        const int s = i % NST, key0 = (chunk0 + i) * C;
        const unsigned char* Ks = smem + s * STAGE;
        cp_async_wait<NST - 1>();
        __syncthreads();

        // phase 1: s = q.k -- warp w: keys 8w..8w+7 against every tile of 16 queries
#pragma unroll
        for (int t = 0; t < QT; ++t) {
            const int qt = 16 * t;
            if (qt < Qpad) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                const unsigned char* qa = Qb + (qt + g8) * KROW + 16 * t4;
                const unsigned char* kb = Ks + (8 * warp + g8) * KROW + 16 * t4;
#pragma unroll
                for (int j = 0; j < HD / 32; ++j) {
                    const uint4 A0 = *reinterpret_cast<const uint4*>(qa + 64 * j);
                    const uint4 A1 = *reinterpret_cast<const uint4*>(qa + 8 * KROW + 64 * j);
                    const uint4 Bk = *reinterpret_cast<const uint4*>(kb + 64 * j);
                    mma_bf16_16816(c, A0.x, A1.x, A0.y, A1.y, Bk.x, Bk.y);
                    mma_bf16_16816(c, A0.z, A1.z, A0.w, A1.w, Bk.z, Bk.w);
                }
                float* sp = S + (size_t)(qt + g8) * SP + 8 * warp + 2 * t4;
                *reinterpret_cast<float2*>(sp) = make_float2(c[0], c[1]);
                *reinterpret_cast<float2*>(sp + 8 * SP) = make_float2(c[2], c[3]);
            }
        }
        __syncthreads();

        // phase 2: one warp per query: scale, mask, the online-softmax update of (max, sum) over
        // the chunk's 64 keys; p goes to Pb as bf16 (zeros for the padding rows of the last tile)
        for (int qi = warp; qi < Qpad; qi += T / 32) {
            uint16_t* pb = reinterpret_cast<uint16_t*>(Pb + (size_t)qi * PBROW);
            if (qi >= Q) {
                pb[lane] = 0;
                pb[lane + 32] = 0;
                if (lane == 0) Alpha[qi] = 1.f;
                continue;
            }
            const int pos = pos0 + qi / G;
            float s0 = S[(size_t)qi * SP + lane] * scale;
            float s1 = S[(size_t)qi * SP + lane + 32] * scale;
            if (key0 + lane > pos) s0 = -INFINITY;
            if (key0 + lane + 32 > pos) s1 = -INFINITY;
            float mx = fmaxf(s0, s1);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float m_old = Mrun[qi];
            const float m_new = fmaxf(m_old, mx);
            // no key of this row seen yet (m_new = -inf): nothing changes
            const float alpha = (m_new == -INFINITY) ? 1.f : expf(m_old - m_new);
            const float p0 = (s0 == -INFINITY) ? 0.f : expf(s0 - m_new);
            const float p1 = (s1 == -INFINITY) ? 0.f : expf(s1 - m_new);
            float l = p0 + p1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            pb[lane] = f2bf(p0);
            pb[lane + 32] = f2bf(p1);
            if (lane == 0) {
                Mrun[qi] = m_new;
                Lrun[qi] = fmaf(Lrun[qi], alpha, l);
                Alpha[qi] = alpha;
            }
        }
        __syncthreads();

        // phase 3: o = o * alpha + p.v -- warp w: its output dims for every tile of 16 queries
        {
            const uint32_t vlane = smem0 + (uint32_t)(s * STAGE) + C * KROW + vlane_off;
#pragma unroll
            for (int t = 0; t < QT; ++t) {
                const int qt = 16 * t;
                if (qt < Qpad) {
                    const float a_lo = Alpha[qt + g8], a_hi = Alpha[qt + g8 + 8];
#pragma unroll
                    for (int nt = 0; nt < NTW; ++nt) {
                        acc[t][nt][0] *= a_lo;
                        acc[t][nt][1] *= a_lo;
                        acc[t][nt][2] *= a_hi;
                        acc[t][nt][3] *= a_hi;
                    }
                    const unsigned char* pa = Pb + (size_t)(qt + g8) * PBROW + 4 * t4;
#pragma unroll
                    for (int kk = 0; kk < C / 16; ++kk) {
                        const uint32_t a0 = *reinterpret_cast<const uint32_t*>(pa + 32 * kk);
                        const uint32_t a1 = *reinterpret_cast<const uint32_t*>(pa + 8 * PBROW + 32 * kk);
                        const uint32_t a2 = *reinterpret_cast<const uint32_t*>(pa + 32 * kk + 16);
                        const uint32_t a3 = *reinterpret_cast<const uint32_t*>(pa + 8 * PBROW + 32 * kk + 16);
                        uint32_t r0, r1, r2, r3;
                        ldmatrix_x4_trans(vlane + (uint32_t)(16 * kk * VROW), r0, r1, r2, r3);
                        mma_bf16_16816(acc[t][0], a0, a1, a2, a3, r0, r1);
                        if (NTW == 2) mma_bf16_16816(acc[t][NTW - 1], a0, a1, a2, a3, r2, r3);
                    }
                }
            }
        }
        __syncthreads();  // everybody is done with stage s: refill it with the chunk NST further on
        if (i + NST < nc) stage_rows(chunk0 + i + NST, s, 0, last_pos, (chunk0 + i + NST) * C + C - 1);
        cp_async_commit();
    }
    cp_async_wait<0>();

    // this span's un-normalised values, for the whole cluster to read
    if (nc > 0) {
#pragma unroll
        for (int t = 0; t < QT; ++t) {
            const int qt = 16 * t;
            if (qt < Qpad) {
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt) {
                    float* dst = Om + (size_t)(qt + g8) * HD + d0 + 8 * nt + 2 * t4;
                    *reinterpret_cast<float2*>(dst) = make_float2(acc[t][nt][0], acc[t][nt][1]);
                    *reinterpret_cast<float2*>(dst + 8 * HD) = make_float2(acc[t][nt][2], acc[t][nt][3]);
                }
            }
        }
    }
    cluster_sync_all();

    // Combine: CTA k < n_active takes an equal share of the (query, pair of dims) outputs and
    // adds the spans that the query's row can see, in span order: weights exp(max_j - max),
    // denominator and values summed j = 0, 1, ...  -- an order fixed by the row's position.
    if (rank < n_active) {
        const int total = Q * (HD / 2);
        const int per = (total + n_active - 1) / n_active;
        const int hi = min(total, (rank + 1) * per);
        const uint32_t om0 = smem0, m0 = (uint32_t)__cvta_generic_to_shared(Mrun),
                       l0 = (uint32_t)__cvta_generic_to_shared(Lrun);
        for (int pp = rank * per + tid; pp < hi; pp += T) {
            const int qi = pp / (HD / 2), dp = pp % (HD / 2);
            const int m = qi / G, g = qi % G;
            const int nk = (pos0 + m) / (C * span_chunks) + 1;  // spans this row sees (<= n_active)
            float mj[kAttnMaxCluster], lj[kAttnMaxCluster];
            float2 oj[kAttnMaxCluster];
#pragma unroll
            for (int j = 0; j < kAttnMaxCluster; ++j) {
                if (j < nk) {
                    mj[j] = ld_cluster_f(cluster_map(m0 + 4 * qi, j));
                    lj[j] = ld_cluster_f(cluster_map(l0 + 4 * qi, j));
                    oj[j] = ld_cluster_f2(cluster_map(om0 + 4 * (qi * HD + 2 * dp), j));
                }
            }
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < kAttnMaxCluster; ++j)
                if (j < nk) mx = fmaxf(mx, mj[j]);
            float l = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
            for (int j = 0; j < kAttnMaxCluster; ++j) {
                if (j < nk) {
                    const float w = expf(mj[j] - mx);
                    l = fmaf(lj[j], w, l);
                    o0 = fmaf(oj[j].x, w, o0);
                    o1 = fmaf(oj[j].y, w, o1);
                }
            }
            *reinterpret_cast<uint32_t*>(out + ((size_t)m * Hq + (size_t)kh * G + g) * HD + 2 * dp) =
                pack_bf16(o0 / l, o1 / l);
        }
    }
    cluster_sync_all();  // nobody leaves while its shared memory may still be read
}

}  // namespace ls

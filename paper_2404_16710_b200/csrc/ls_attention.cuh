// Decode / verify attention over the paged bf16 KV cache (one KV cache shared by the draft
// and the verify stage, LayerSkip Sec. 4.3.3), for passes of up to 16 rows.
//
// One thread-block cluster of S CTAs per KV head.  The keys are cut by ABSOLUTE position into
// chunks of 64; CTA k of the cluster owns the chunks k, k + S, k + 2S, ... (its "span"), streams
// them through a two-stage cp.async ring and keeps a running (max, sum, weighted values) per
// query -- the online-softmax recurrence, chunk after chunk in position order.  The spans'
// results never go through global memory: every CTA leaves (max, sum, values) in its own shared
// memory, the cluster meets at a barrier, and each CTA then combines a slice of the
// (query, dim) outputs by reading all spans through distributed shared memory, in span order.
// No counters, no fences, no second kernel.
//
// Which CTA takes a chunk depends on the chunk's position and on S, a constant of the model's
// head layout, so what a row's result depends on is its position alone -- not the pass size,
// not the cache capacity, not the other sequences of a pass: a chunk that lies wholly beyond
// the row's position leaves its running state bit for bit as it was (weights 0, scale factor
// exp(0)), which makes the verify pass of d+1 rows (Sec. 4.3.2) reproduce single-token decoding
// exactly.  Dealing the chunks out round-robin also keeps the CTAs evenly loaded at any length.
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

// launch shape of the attention kernel for one model: CTAs per cluster
struct AttnPlan {
    int csize;
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
// shared memory: stage[2] { Ks [64][HD*2+64 B] | Vs [64][HD*2+16 B] } | Qb bf16 [Qpad][HD*2+64 B]
//   | Pb bf16 [Qpad][72] | Wmax, Wsum f32 [Qpad][8] (per-warp row maxima and sums of a chunk)
//   | Mrun f32 [2][Qpad] | Lrun, Alpha f32 [Qpad] | Rml float2 [8][Qpad] | Ro float2 [Q HD/2 + 8]
// (Qpad = Q rounded up to 16).  Rml and Ro are written by the OTHER CTAs of the cluster: span j
// sends its (max, sum) per query and, to the CTA that combines them, its un-normalised values.
template <int HD>
__host__ __device__ constexpr size_t attn_stage_bytes()
{
    return (size_t)kAttnChunk * (HD * 2 + 64) + (size_t)kAttnChunk * (HD * 2 + 16);
}
template <int HD>
__host__ __device__ constexpr size_t attn_smem_bytes(int Q)
{
    const size_t qpad = ((size_t)Q + 15) / 16 * 16;
    return kAttnStages * attn_stage_bytes<HD>() + qpad * (HD * 2 + 64) + qpad * kAttnSP * 2 +
           sizeof(float) * qpad * (8 + 8 + 2 + 1 + 1) + sizeof(float2) * (kAttnMaxCluster * qpad + (size_t)Q * (HD / 2) + 8);
}

// n / d for small operands without the integer-division sequence: mul = ceil(2^32 / d) (any value
// for d == 1); exact while n * d < 2^32
__device__ __forceinline__ uint32_t fastdiv_mul(uint32_t d) { return d > 1 ? 0xffffffffu / d + 1u : 0u; }
__device__ __forceinline__ int fastdiv(int n, int d, uint32_t mul) { return d == 1 ? n : (int)__umulhi((uint32_t)n, mul); }

__device__ __forceinline__ void st_cluster_f2(uint32_t addr, float a, float b)
{
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1,%2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
// an arrival that orders no memory accesses ("this CTA has started")
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// grid (cluster size, Hkv, sequences), cluster (cluster size, 1, 1), block 256.  QT: tiles of 16
// queries the instantiation can hold (Q = G * rows per sequence <= 16 QT).
// With several sequences per pass (gridDim.z = B; M counts all rows) the cluster of sequence b
// takes the rows r = m B + b, that sequence's control block and its page-table entries
// (b * pt_stride ..); max_seq is then the capacity of one sequence.
template <int HD, int QT>
__global__ void __launch_bounds__(kAttnThreads)
attn_cluster_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ kpages,
                    const uint16_t* __restrict__ vpages, const int32_t* __restrict__ page_table,
                    int32_t* ctl, int pos_off, int M, int Hq, int Hkv, int page_shift,
                    int max_seq, uint16_t* __restrict__ out, int gate, int pt_stride)
{
    constexpr int C = kAttnChunk, T = kAttnThreads, NST = kAttnStages;
    constexpr int KROW = HD * 2 + 64, VROW = HD * 2 + 16;
    constexpr int PBROW = kAttnSP * 2;
    constexpr int SEGS = HD * 2 / 16;  // 16-byte segments per row
    constexpr int NTW = HD / 64;       // n8 tiles of output dims per warp: 2 (HD 128) or 1 (HD 64)
    constexpr int HP = HD / 2;         // pairs of dims per query
    constexpr size_t STAGE = attn_stage_bytes<HD>();
    static_assert(STAGE % 16 == 0, "stages keep 16-byte alignment");
    extern __shared__ __align__(16) unsigned char smem[];
    const int kh = blockIdx.y, tid = threadIdx.x;
    const int nseq = (int)gridDim.z, sq = (int)blockIdx.z;
    const int32_t* sctl = ctl ? ctl + sq * CTL_WORDS : nullptr;  // this sequence's control words
    page_table += sq * pt_stride;
    M /= nseq;  // rows of this sequence
    const int rank = (int)cluster_ctarank(), csize = (int)gridDim.x;
    const int warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    auto chunk_of = [&](int i) { return rank + i * csize; };  // i-th chunk of this CTA's span
    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(smem);
    const bool one_page = page_shift >= 6;  // a chunk never straddles a page of 64 tokens or more

    // chunk c into stage s: rows up to position p_hi are copied, the rest of the chunk is zeroed.
    // A thread moves the same 16-byte segment of rows r0, r0 + T/SEGS, ...
    const int seg = tid % SEGS, r0 = tid / SEGS;
    // (phys: the physical page of the chunk's first key, looked up by the caller ahead of time when
    // chunks do not straddle pages)
    auto chunk_page = [&](int c) { return one_page ? page_table[(c * C) >> page_shift] : 0; };
    auto stage_chunk = [&](int c, int s, int p_hi, int phys) {
        const int key0 = c * C;
        uint32_t kd = smem0 + (uint32_t)(s * STAGE) + r0 * KROW + seg * 16;
        uint32_t vd = smem0 + (uint32_t)(s * STAGE) + C * KROW + r0 * VROW + seg * 16;
        if (one_page) {
            const size_t off = ((((size_t)phys * Hkv + kh) << page_shift) + (key0 & ((1 << page_shift) - 1)) + r0) * HD + seg * 8;
            const uint16_t *ks = kpages + off, *vs = vpages + off;
            const int n_ok = p_hi - key0 - r0;  // rows r0 + j T/SEGS with j T/SEGS <= n_ok exist
#pragma unroll
            for (int it = 0; it < C * SEGS / T; ++it) {
                const int nb = it * (T / SEGS) <= n_ok ? 16 : 0;
                cp_async16_cg(kd, ks, nb);
                cp_async16_cg(vd, vs, nb);
                kd += (T / SEGS) * KROW;
                vd += (T / SEGS) * VROW;
                ks += (T / SEGS) * HD;
                vs += (T / SEGS) * HD;
            }
        } else {
#pragma unroll
            for (int it = 0; it < C * SEGS / T; ++it) {
                const int p = key0 + r0 + it * (T / SEGS);
                const bool ok = p <= p_hi;
                const size_t off = kv_row_offset(page_table, ok ? p : key0, page_shift, Hkv, kh, HD) + seg * 8;
                cp_async16_cg(kd, kpages + off, ok ? 16 : 0);
                cp_async16_cg(vd, vpages + off, ok ? 16 : 0);
                kd += (T / SEGS) * KROW;
                vd += (T / SEGS) * VROW;
            }
        }
    };

    // Cache rows below the loop's cache length do not change while the loop runs, so the first
    // chunks of the span that lie wholly below it are fetched before the producer of q (and of
    // this pass's own k, v rows) has finished.  The length is read past L1 and may be an older,
    // smaller one: then fewer chunks go early.
    TR_T0
    pdl_launch_dependents();
    cluster_arrive_relaxed();  // "this CTA runs": waited for before the first write into another CTA's memory
    int phys0[NST];  // the page table does not change while a loop runs: look the first chunks up at once
#pragma unroll
    for (int s = 0; s < NST; ++s) phys0[s] = chunk_of(s) * C < max_seq ? chunk_page(chunk_of(s)) : 0;
    int c_early = 0;
    if (ctl && !(gate > 0 && gate > __ldcg(ctl + CTL_D_EFF))) c_early = min(__ldcg(sctl + CTL_CACHE_LEN), max_seq);
    bool early[NST];
#pragma unroll
    for (int s = 0; s < NST; ++s) {
        early[s] = (chunk_of(s) + 1) * C <= c_early;
        if (early[s]) stage_chunk(chunk_of(s), s, c_early - 1, phys0[s]);
    }
    pdl_wait();
    TR_T1
    auto leave = [&]() {  // nothing in flight may outlive the CTA's shared memory; every arrive gets its wait
        cp_async_commit();
        cp_async_wait<0>();
        cluster_wait();
    };
    // the two ways out below are taken by every CTA of the grid alike (they depend on the
    // control words and the launch arguments only), so no CTA is left waiting at a cluster barrier
    if (pass_idle(ctl, gate)) return leave();
    const int pos0 = (ctl ? sctl[CTL_CACHE_LEN] : 0) + pos_off;
    const int last_pos = pos0 + M - 1;
    const int G = Hq / Hkv, Q = G * M;  // query qi = m * G + g
    const int Qpad = (Q + 15) & ~15;
    if (last_pos >= max_seq || pos0 < 0 || Qpad > 16 * QT) {
        if (ctl && tid == 0) ctl[CTL_STATUS] = DEV_POS_OVERFLOW;
        return leave();
    }
    // (an early chunk lies below a cache length that only grows: below pos0, all of it visible)
    const int last_chunk = last_pos / C;
    const int n_active = min(csize, last_chunk + 1);  // spans with a visible key
    // chunks this CTA walks: its span, cut at the last visible key
    const int nc = rank <= last_chunk ? (last_chunk - rank) / csize + 1 : 0;

    unsigned char* Qb = smem + NST * STAGE;
    unsigned char* Pb = Qb + (size_t)Qpad * KROW;
    float* Wmax = reinterpret_cast<float*>(Pb + (size_t)Qpad * PBROW);  // [Qpad][8]
    float* Wsum = Wmax + Qpad * 8;                                      // [Qpad][8]
    float* Mrun = Wsum + Qpad * 8;                                      // [2][Qpad]: read one, write the other
    float* Lrun = Mrun + 2 * Qpad;
    float* Alpha = Lrun + Qpad;
    float2* Rml = reinterpret_cast<float2*>(Alpha + Qpad);              // [8][Qpad] (max, sum) of span j
    float2* Ro = Rml + kAttnMaxCluster * Qpad;                          // [n_active][per] values of span j

    const uint32_t gmul = fastdiv_mul((uint32_t)G);
    // the group's queries (16-byte pieces, zeros for the padding rows) travel with the first chunk
    if (nc > 0) {
        const uint32_t qb0 = smem0 + (uint32_t)(NST * STAGE);
        for (int qi = r0; qi < Qpad; qi += T / SEGS) {
            const int m = qi < Q ? fastdiv(qi, G, gmul) : 0, g = qi < Q ? qi - m * G : 0;
            cp_async16_ca(qb0 + qi * KROW + seg * 16, q + ((size_t)(m * nseq + sq) * Hq + (size_t)kh * G + g) * HD + seg * 8,
                          qi < Q ? 16 : 0);
        }
    }
    // the first chunks that did not go early (zeros beyond the last visible key), one commit
    // group per chunk slot, empty when the span has no such chunk
#pragma unroll
    for (int s = 0; s < NST; ++s) {
        if (s < nc && !early[s]) stage_chunk(chunk_of(s), s, last_pos, phys0[s]);
        cp_async_commit();
    }
    for (int qi = tid; qi < Qpad; qi += T) {
        Mrun[qi] = -INFINITY;
        Lrun[qi] = 0.f;
    }
    // p of the padding rows stays zero: rows 8..15 of a tile are skipped where none of them is a query
    for (int idx = tid; idx < Qpad * (PBROW / 16); idx += T) reinterpret_cast<uint4*>(Pb)[idx] = make_uint4(0, 0, 0, 0);

    float acc[QT][NTW][4];
#pragma unroll
    for (int t = 0; t < QT; ++t)
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[t][nt][i] = 0.f;

    // position of the thread's two rows in every tile of queries (-1: a padding row, sees no key)
    int rowpos[QT][2];
#pragma unroll
    for (int t = 0; t < QT; ++t)
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {
            const int qi = 16 * t + g8 + 8 * hrow;
            rowpos[t][hrow] = qi < Q ? pos0 + fastdiv(qi, G, gmul) : -1;
        }
    const float scale = rsqrtf((float)HD);
    const int d0 = NTW * 8 * warp;  // this warp's output dims in p.v
    // ldmatrix: lane L addresses row L%8 of matrix L/8; matrices 0, 1: keys 0-7, 8-15 of the
    // 16-key block at dims d0..d0+7; matrices 2, 3: the same keys at dims d0+8..
    const int mi = lane >> 3, mr = lane & 7;
    const uint32_t vlane_off = (uint32_t)(((mi & 1) * 8 + mr) * VROW + (d0 + ((NTW == 2) ? (mi >> 1) * 8 : 0)) * 2);

    uint4 qf0[HD / 32], qf1[HD / 32];
    for (int i = 0; i < nc; ++i) {
        const int s = i % NST, key0 = chunk_of(i) * C;
        const unsigned char* Ks = smem + s * STAGE;
        const float* Mold = Mrun + (i & 1) * Qpad;
        float* Mnew = Mrun + ((i + 1) & 1) * Qpad;
        const int phys_next = i + NST < nc ? chunk_page(chunk_of(i + NST)) : 0;
        cp_async_wait<NST - 1>();
        __syncthreads();
        if (QT == 1 && i == 0) {  // a single tile of queries: its fragments stay in registers
            const unsigned char* qa = Qb + g8 * KROW + 16 * t4;
#pragma unroll
            for (int j = 0; j < HD / 32; ++j) {
                qf0[j] = *reinterpret_cast<const uint4*>(qa + 64 * j);
                qf1[j] = *reinterpret_cast<const uint4*>(qa + 8 * KROW + 64 * j);
            }
        }

        // phase A: scores of the warp's keys 8w..8w+7 against every tile of 16 queries, kept in
        // registers (rows g8 and g8+8 of the tile, keys 8w+2t4 and +1), scaled and masked; the
        // warp's maximum per row goes to Wmax
        float sc[QT][4];
#pragma unroll
        for (int t = 0; t < QT; ++t) {
            const int qt = 16 * t;
            if (qt < Qpad) {
                float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
                const unsigned char* qa = Qb + (qt + g8) * KROW + 16 * t4;
                const unsigned char* kb = Ks + (8 * warp + g8) * KROW + 16 * t4;
#pragma unroll
                for (int j = 0; j < HD / 32; ++j) {
                    const uint4 A0 = QT == 1 ? qf0[j] : *reinterpret_cast<const uint4*>(qa + 64 * j);
                    const uint4 A1 = QT == 1 ? qf1[j] : *reinterpret_cast<const uint4*>(qa + 8 * KROW + 64 * j);
                    const uint4 Bk = *reinterpret_cast<const uint4*>(kb + 64 * j);
                    mma_bf16_16816(c0, A0.x, A1.x, A0.y, A1.y, Bk.x, Bk.y);
                    mma_bf16_16816(c1, A0.z, A1.z, A0.w, A1.w, Bk.z, Bk.w);
                }
                const int key = key0 + 8 * warp + 2 * t4;
                const bool upper = qt + 8 < Q;  // rows 8..15 of the tile hold a query (the same for all threads)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    sc[t][e] = (key + (e & 1) <= rowpos[t][e >> 1]) ? (c0[e] + c1[e]) * scale : -INFINITY;
                float mlo = fmaxf(sc[t][0], sc[t][1]);
                mlo = fmaxf(mlo, __shfl_xor_sync(0xffffffffu, mlo, 1));
                mlo = fmaxf(mlo, __shfl_xor_sync(0xffffffffu, mlo, 2));
                if (t4 == 0) Wmax[(qt + g8) * 8 + warp] = mlo;
                if (upper) {
                    float mhi = fmaxf(sc[t][2], sc[t][3]);
                    mhi = fmaxf(mhi, __shfl_xor_sync(0xffffffffu, mhi, 1));
                    mhi = fmaxf(mhi, __shfl_xor_sync(0xffffffffu, mhi, 2));
                    if (t4 == 0) Wmax[(qt + g8 + 8) * 8 + warp] = mhi;
                }
            }
        }
        __syncthreads();

        // phase B: every thread, for its two rows: chunk maximum (the 8 warps' maxima in warp
        // order), the online-softmax step of the running maximum, p = exp(s - max) for its four
        // scores; p goes to Pb as bf16, the warp's sum per row to Wsum
        float alpha[QT][2];
#pragma unroll
        for (int t = 0; t < QT; ++t) {
            const int qt = 16 * t;
            if (qt < Qpad) {
#pragma unroll
                for (int hrow = 0; hrow < 2; ++hrow) {
                    const int qi = qt + g8 + 8 * hrow;
                    if (hrow == 1 && !(qt + 8 < Q)) {  // no query in rows 8..15: their p stays zero
                        alpha[t][1] = 1.f;
                        continue;
                    }
                    const float4 w0 = *reinterpret_cast<const float4*>(Wmax + qi * 8);
                    const float4 w1 = *reinterpret_cast<const float4*>(Wmax + qi * 8 + 4);
                    const float mc = fmaxf(fmaxf(fmaxf(w0.x, w0.y), fmaxf(w0.z, w0.w)), fmaxf(fmaxf(w1.x, w1.y), fmaxf(w1.z, w1.w)));
                    const float m_old = Mold[qi];
                    const float m_new = fmaxf(m_old, mc);
                    // no key of this row seen yet (m_new = -inf): nothing changes
                    const float al = (m_new == -INFINITY) ? 1.f : __expf(m_old - m_new);
                    const float s0 = sc[t][2 * hrow], s1 = sc[t][2 * hrow + 1];
                    const float p0 = (s0 == -INFINITY) ? 0.f : __expf(s0 - m_new);
                    const float p1 = (s1 == -INFINITY) ? 0.f : __expf(s1 - m_new);
                    float l = p0 + p1;
                    l += __shfl_xor_sync(0xffffffffu, l, 1);
                    l += __shfl_xor_sync(0xffffffffu, l, 2);
                    *reinterpret_cast<uint32_t*>(Pb + (size_t)qi * PBROW + (8 * warp + 2 * t4) * 2) = pack_bf16(p0, p1);
                    if (t4 == 0) Wsum[qi * 8 + warp] = l;
                    if (warp == 0 && t4 == 0) {
                        Mnew[qi] = m_new;
                        Alpha[qi] = al;
                    }
                    alpha[t][hrow] = al;
                }
            }
        }
        __syncthreads();

        // phase C: o = o * alpha + p.v -- warp w: its output dims for every tile of 16 queries;
        // one thread per query adds the warps' sums, in warp order, to the running sum
        if (tid < Q) {
            const float4 w0 = *reinterpret_cast<const float4*>(Wsum + tid * 8);
            const float4 w1 = *reinterpret_cast<const float4*>(Wsum + tid * 8 + 4);
            const float l = ((((((w0.x + w0.y) + w0.z) + w0.w) + w1.x) + w1.y) + w1.z) + w1.w;
            Lrun[tid] = fmaf(Lrun[tid], Alpha[tid], l);
        }
        {
            const uint32_t vlane = smem0 + (uint32_t)(s * STAGE) + C * KROW + vlane_off;
#pragma unroll
            for (int t = 0; t < QT; ++t) {
                const int qt = 16 * t;
                if (qt < Qpad) {
#pragma unroll
                    for (int nt = 0; nt < NTW; ++nt) {
                        acc[t][nt][0] *= alpha[t][0];
                        acc[t][nt][1] *= alpha[t][0];
                        acc[t][nt][2] *= alpha[t][1];
                        acc[t][nt][3] *= alpha[t][1];
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
        if (i + NST < nc) {
            __syncthreads();  // everybody is done with stage s: refill it with the chunk NST further on
            stage_chunk(chunk_of(i + NST), s, last_pos, phys_next);
        }
        cp_async_commit();
    }
    cp_async_wait<0>();
    __syncthreads();  // the running maxima and sums are final

    // Combine.  The (query, pair of dims) outputs are dealt out in equal shares to the CTAs
    // k < n_active; span j sends each owner its un-normalised values of the owner's share, and
    // every owner its (max, sum) per query -- for the rows that can see span j at all.
    const int total = Q * HP;
    const int per = (total + n_active - 1) / n_active;
    const uint32_t pmul = fastdiv_mul((uint32_t)per);
    cluster_wait();  // every CTA of the cluster runs: its shared memory may be written
    if (nc > 0) {
        const float* Mfin = Mrun + (nc & 1) * Qpad;
        const uint32_t ro0 = (uint32_t)__cvta_generic_to_shared(Ro), rml0 = (uint32_t)__cvta_generic_to_shared(Rml);
#pragma unroll
        for (int t = 0; t < QT; ++t) {
#pragma unroll
            for (int hrow = 0; hrow < 2; ++hrow) {
                const int qi = 16 * t + g8 + 8 * hrow;
                if (rowpos[t][hrow] >= rank * C) {  // the row sees this span's first chunk (padding rows: -1)
#pragma unroll
                    for (int nt = 0; nt < NTW; ++nt) {
                        const int pp = qi * HP + (d0 + 8 * nt) / 2 + t4;
                        const int k = fastdiv(pp, per, pmul);
                        st_cluster_f2(cluster_map(ro0 + 8u * (uint32_t)(rank * per + pp - k * per), k),
                                      acc[t][nt][2 * hrow], acc[t][nt][2 * hrow + 1]);
                    }
                }
            }
        }
        for (int idx = tid; idx < Q * kAttnMaxCluster; idx += T) {
            const int qi = idx / kAttnMaxCluster, k = idx % kAttnMaxCluster;
            if (k < n_active && pos0 + fastdiv(qi, G, gmul) >= rank * C)
                st_cluster_f2(cluster_map(rml0 + 8u * (uint32_t)(rank * Qpad + qi), k), Mfin[qi], Lrun[qi]);
        }
    }
    cluster_arrive();
    cluster_wait();  // everything sent to this CTA has arrived; from here on it reads only its own memory
    if (rank < n_active) {
        // spans in order j = 0, 1, ...: weights exp(max_j - max), denominator and values -- an
        // order fixed by the row's position
        const int hi = min(total, (rank + 1) * per);
        for (int pp = rank * per + tid; pp < hi; pp += T) {
            const int qi = pp / HP, dp = pp % HP;
            const int m = fastdiv(qi, G, gmul), g = qi - m * G;
            const int nk = min(csize, ((pos0 + m) >> 6) + 1);  // spans this row sees (<= n_active)
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < kAttnMaxCluster; ++j)
                if (j < nk) mx = fmaxf(mx, Rml[j * Qpad + qi].x);
            float l = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
            for (int j = 0; j < kAttnMaxCluster; ++j) {
                if (j < nk) {
                    const float2 ml = Rml[j * Qpad + qi];
                    const float2 o = Ro[j * per + pp - rank * per];
                    const float w = __expf(ml.x - mx);
                    l = fmaf(ml.y, w, l);
                    o0 = fmaf(o.x, w, o0);
                    o1 = fmaf(o.y, w, o1);
                }
            }
            *reinterpret_cast<uint32_t*>(out + ((size_t)(m * nseq + sq) * Hq + (size_t)kh * G + g) * HD + 2 * dp) =
                pack_bf16(__fdividef(o0, l), __fdividef(o1, l));
        }
    }
    TR_END(kpages, M > 1 ? 1 : 0)
}

}  // namespace ls

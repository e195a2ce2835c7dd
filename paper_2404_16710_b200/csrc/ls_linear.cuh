// Weight-streaming linear layers for M <= 16 rows: y[m, n] = sum_k W[n, k] h[m, k].
//
// Batch-1 decoding reads every weight byte once per pass and does 2*M flops per weight
// element, so these kernels are HBM-bound; their job is to keep enough 16-byte loads in
// flight and to spend few issue slots per byte.  Two families, chosen per model:
//
//   FMA  one warp per 4 weight rows, lanes stride over K with 128-bit loads, fp32 FMA
//        chains per (row, token), butterfly reduction.  Cheap for M <= 4.
//   MMA  one CTA per 16 weight rows, its 8 or 16 warps interleave over K; a thread's
//        16-byte pieces of the weight rows ARE its mma.sync.m16n8k16 A fragments (the
//        contraction index may be permuted freely as long as A and B agree), so they
//        need no layout change: each thread streams its own pieces through a private
//        cp.async ring in shared memory.  Tokens are the n8 dimension.  Issue cost per
//        weight byte does not grow with M up to 8 (16 with a second n-tile).
//
// In both, the sequence of operations that produces (row n, token m) is the same for
// every M, so results are bit-identical across pass sizes within a family.
//
// Epilogues: plain store, residual add (x <- x + W h, Sec. 4.1 of the paper), SwiGLU
// (gate and up rows of one feature meet in one thread), q|k|v with rotary embedding and
// KV append (the two halves of a rotary pair meet in one thread), LM head + argmax candidates
// (Sec. 2.1 / 4.2: the shared head g; greedy decoding needs only the index).
#pragma once
#include "ls_kernels.cuh"

namespace ls {

enum Epi : int { EPI_STORE = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2, EPI_ARGMAX = 3, EPI_QKV = 4 };

struct LinArgs {
    const uint16_t* w0;  // row segments: rows [0, n0) of w0, then n1 rows of w1, the rest of w2
    const uint16_t* w1;  // (QKV as one launch); SwiGLU: w0 = gate, w1 = up
    const uint16_t* w2;
    int n0, n1;
    const uint16_t* h;   // [M][K] bf16
    int M, N, K;         // N: output rows (SwiGLU: features F)
    float* out;          // fp32 [M][ldo]: store / residual / optional logits
    int ldo;
    uint16_t* out_bf16;  // SwiGLU result [M][N]
    ValIdx* cand;        // argmax candidates [M][cand_stride], one per CTA
    int cand_stride;
    float* second;       // optional [M][cand_stride]: the CTA's second-largest logit (adaptive drafting)
    int32_t* ctl;
    int gate;            // > 0: the launch belongs to draft pass `gate` and idles once drafting has stopped
    // EPI_QKV: rotary embedding + KV append fused behind the q|k|v projection
    const float* inv_freq;       // [hd/2], or nullptr: theta^(-2j/hd) computed in place
    const int32_t* page_table;
    uint16_t *q_out, *kpages, *vpages;
    int Hq, Hkv, hd, page_shift, max_seq, pos_off;
    int nseq, pt_stride;         // sequences sharing the pass (row m: sequence m % nseq) and page-table entries per sequence
    float theta;
    // RMSNorm carried across kernel boundaries.  A producer (residual epilogue, embedding)
    // leaves, beside the fp32 row x, the bf16 row x*gain of its consumer's norm and adds the
    // squares of its own columns to the row's exact sum (ls_common.cuh); a consumer reads those
    // rows as h and scales its accumulators by 1/sqrt(mean x^2 + eps): W (x g) r = W (x r g).
    // The sums of the two norms of a layer live in two arrays; a consumer clears the rows of
    // the array its successor's producer will add to.
    const long long* ss_in;  // consumer: [M][kSsSlots] sums of squares; nullptr: no scaling
    long long* ss_out;       // EPI_RESIDUAL: [M][kSsSlots] sums this launch adds to (cleared beforehand)
    long long* ss_clear;     // consumer: [M][kSsSlots] sums to clear for the next producer, or nullptr
    float inv_d, eps;
    const uint16_t *gain_a, *gain_b;  // EPI_RESIDUAL: hout_x[m * N + n] = bf16(x_new[m][n] * gain_x[n])
    uint16_t *hout_a, *hout_b;
};

// EPI_QKV tiles pair row j of a head with row j + hd/2, the two halves of one rotary pair:
// tile b covers pairs j = 8 (b % (hd/16)) .. +7 of head b / (hd/16).
__device__ __forceinline__ int qkv_row(const LinArgs& a, int tile, int pair, int hi)
{
    const int tph = a.hd >> 4;
    return (tile / tph) * a.hd + (tile % tph) * 8 + pair + (hi ? (a.hd >> 1) : 0);
}

// rotation of pair j at position pos: (sin, cos) of pos * theta^(-2j/hd)
__device__ __forceinline__ void qkv_rotation(const LinArgs& a, int j, int pos, float& sn, float& cs)
{
    const float f = a.inv_freq ? a.inv_freq[j] : (float)pow((double)a.theta, -2.0 * (double)j / (double)a.hd);
    sincosf((float)pos * f, &sn, &cs);
}

// position of row m of the pass: its sequence's cache length + the launch's offset + its row
// within the sequence (one sequence: cache length + offset + m)
__device__ __forceinline__ int row_pos(const LinArgs& a, int m)
{
    if (a.nseq <= 1) return (a.ctl ? a.ctl[CTL_CACHE_LEN] : 0) + a.pos_off + m;
    const int j = m / a.nseq, b = m - j * a.nseq;
    return a.ctl[b * CTL_WORDS + CTL_CACHE_LEN] + a.pos_off + j;
}

// rotate the pair (x_j, x_{j+hd/2}) of head `head` for token m and store it: q -> q_out,
// k, v -> the paged cache row of the row's position in its sequence's pages (v is not rotated)
__device__ __forceinline__ void qkv_store(const LinArgs& a, int head, int j, int m, int pos, float lo, float hi,
                                          float sn, float cs)
{
    const int32_t* page_table = a.page_table + (a.nseq > 1 ? (m % a.nseq) * a.pt_stride : 0);
    if (pos < 0 || pos >= a.max_seq) {
        if (a.ctl) a.ctl[CTL_STATUS] = DEV_POS_OVERFLOW;
        return;
    }
    if (head < a.Hq + a.Hkv) {
        const float r0 = lo * cs - hi * sn, r1 = lo * sn + hi * cs;
        lo = r0;
        hi = r1;
    }
    uint16_t* dst;
    if (head < a.Hq) dst = a.q_out + ((size_t)m * a.Hq + head) * a.hd;
    else if (head < a.Hq + a.Hkv) dst = a.kpages + kv_row_offset(page_table, pos, a.page_shift, a.Hkv, head - a.Hq, a.hd);
    else dst = a.vpages + kv_row_offset(page_table, pos, a.page_shift, a.Hkv, head - a.Hq - a.Hkv, a.hd);
    dst[j] = f2bf(lo);
    dst[j + (a.hd >> 1)] = f2bf(hi);
}

__device__ __forceinline__ const uint16_t* weight_row(const LinArgs& a, int n)
{
    n = min(n, a.N - 1);
    if (n < a.n0) return a.w0 + (size_t)n * a.K;
    n -= a.n0;
    if (n < a.n1) return a.w1 + (size_t)n * a.K;
    n -= a.n1;
    return a.w2 + (size_t)n * a.K;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.0f + expf(-g)) * u; }

// =============================================================================== FMA family
// grid ceil(N/16) (SwiGLU: ceil(F/8)), block 128 = 4 warps x 4 weight rows.
template <int MT, int EPI>
__global__ void __launch_bounds__(128) linear_fma_kernel(const LinArgs a)
{
    TR_T0
    pdl_launch_dependents();
    pdl_wait();
    TR_T1
    if (pass_idle(a.ctl, a.gate)) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint16_t* rp[4];
    int nrow[4];  // output index of each of the warp's rows
    if (EPI == EPI_SWIGLU) {
        int f = blockIdx.x * 8 + warp * 2;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            nrow[r] = f + (r & 1);
            int fc = min(nrow[r], a.N - 1);
            rp[r] = ((r < 2) ? a.w0 : a.w1) + (size_t)fc * a.K;
        }
    } else if (EPI == EPI_QKV) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            nrow[r] = qkv_row(a, blockIdx.x, warp * 2 + (r & 1), r >> 1);
            rp[r] = weight_row(a, nrow[r]);
        }
    } else {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            nrow[r] = blockIdx.x * 16 + warp * 4 + r;
            rp[r] = weight_row(a, nrow[r]);
        }
    }
    float acc[4][MT];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[r][m] = 0.f;

    const int nchunks = a.K >> 3;
#pragma unroll 2
    for (int c = lane; c < nchunks; c += 32) {
        float wf[4][8];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            uint4 v = ld_stream16(rp[r] + 8 * c);
            wf[r][0] = bf16lo(v.x); wf[r][1] = bf16hi(v.x);
            wf[r][2] = bf16lo(v.y); wf[r][3] = bf16hi(v.y);
            wf[r][4] = bf16lo(v.z); wf[r][5] = bf16hi(v.z);
            wf[r][6] = bf16lo(v.w); wf[r][7] = bf16hi(v.w);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            uint4 v = ld_reuse16(a.h + (size_t)min(m, a.M - 1) * a.K + 8 * c);
            float xf[8] = {bf16lo(v.x), bf16hi(v.x), bf16lo(v.y), bf16hi(v.y),
                           bf16lo(v.z), bf16hi(v.z), bf16lo(v.w), bf16hi(v.w)};
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float s = acc[r][m];
#pragma unroll
                for (int e = 0; e < 8; ++e) s = fmaf(wf[r][e], xf[e], s);
                acc[r][m] = s;
            }
        }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float v = acc[r][m];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            acc[r][m] = v;
        }

    if (a.ss_in) {  // fused RMSNorm: scale row m by 1/sqrt(mean x^2 + eps)
        __shared__ float rs[kMaxRows];
        for (int m0 = 0; m0 < a.M; m0 += 128 / kSsSlots)  // 128 threads: 8 rows at a time
            rms_rscales(a.ss_in + (size_t)m0 * kSsSlots, a.ss_clear ? a.ss_clear + (size_t)m0 * kSsSlots : nullptr,
                        min(a.M - m0, 128 / kSsSlots), a.inv_d, a.eps, rs + m0);
        __syncthreads();
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float v = rs[min(m, a.M - 1)];
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[r][m] *= v;
        }
    }

    if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
        __shared__ long long sq[4][MT];
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (lane == m) {
                long long q = 0;
                if (m < a.M) {
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        if (nrow[r] < a.N) {
                            float* o = a.out + (size_t)m * a.ldo + nrow[r];
                            const float xn = (EPI == EPI_RESIDUAL) ? (*o + acc[r][m]) : acc[r][m];
                            *o = xn;
                            if (EPI == EPI_RESIDUAL) {
                                q += sq_fixed(xn);
                                if (a.hout_a) a.hout_a[(size_t)m * a.N + nrow[r]] = f2bf(xn * bf16f(a.gain_a[nrow[r]]));
                                if (a.hout_b) a.hout_b[(size_t)m * a.N + nrow[r]] = f2bf(xn * bf16f(a.gain_b[nrow[r]]));
                            }
                        }
                }
                sq[warp][m] = q;
            }
        if (EPI == EPI_RESIDUAL && a.ss_out) {
            __syncthreads();
            if (threadIdx.x < MT && threadIdx.x < a.M) {
                const int m = threadIdx.x;
                ss_add(a.ss_out + (size_t)m * kSsSlots, sq[0][m] + sq[1][m] + sq[2][m] + sq[3][m]);
            }
        }
    } else if (EPI == EPI_SWIGLU) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (lane == m && m < a.M) {
#pragma unroll
                for (int r = 0; r < 2; ++r)
                    if (nrow[r] < a.N)
                        a.out_bf16[(size_t)m * a.N + nrow[r]] = f2bf(silu_mul(acc[r][m], acc[r + 2][m]));
            }
    } else if (EPI == EPI_QKV) {
        const int tph = a.hd >> 4;
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (lane == m && m < a.M) {
                const int pos = row_pos(a, m);
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int j = (blockIdx.x % tph) * 8 + warp * 2 + r;
                    float sn, cs;
                    qkv_rotation(a, j, pos, sn, cs);
                    qkv_store(a, blockIdx.x / tph, j, m, pos, acc[r][m], acc[r + 2][m], sn, cs);
                }
            }
    } else {  // EPI_ARGMAX
        __shared__ float bv[4][MT];
        __shared__ float bs[4][MT];
        __shared__ int bi[4][MT];
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (lane == m) {
                float v = -INFINITY, s2 = -INFINITY;
                int idx = 0x7fffffff;
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if (nrow[r] < a.N) {
                        if (a.out && m < a.M) a.out[(size_t)m * a.ldo + nrow[r]] = acc[r][m];
                        top2_push(acc[r][m], nrow[r], v, idx, s2);
                    }
                bv[warp][m] = v;
                bs[warp][m] = s2;
                bi[warp][m] = idx;
            }
        __syncthreads();
        if (threadIdx.x < MT && threadIdx.x < a.M) {
            int m = threadIdx.x;
            float v = bv[0][m], s2 = bs[0][m];
            int idx = bi[0][m];
#pragma unroll
            for (int w = 1; w < 4; ++w) top2_merge(bv[w][m], bi[w][m], bs[w][m], v, idx, s2);
            ValIdx e;
            e.v = v;
            e.i = idx;
            a.cand[(size_t)m * a.cand_stride + blockIdx.x] = e;
            if (a.second) a.second[(size_t)m * a.cand_stride + blockIdx.x] = s2;
        }
    }
    TR_END(a.w0, a.M > 1 ? 1 : 0)
}

// =============================================================================== MMA family

template <int NT, int TR, int WARPS, int STAGES>
__host__ __device__ constexpr size_t mma_ring_bytes()
{
    return (size_t)(2 * TR + NT) * STAGES * WARPS * 32 * 16;
}

// grid ceil(tiles/TR) with tiles = ceil(N/16) (SwiGLU: ceil(F/8)), block WARPS*32: the warps
// interleave over K in steps of 32.  Fragment roles (g = lane/4, t = lane%4): the thread's
// 16 bytes of row g (and of row g+8) at k = 32 s + 8 t feed two MMAs; contraction slots
// {2t, 2t+1, 2t+8, 2t+9} of the first take elements k..k+3, of the second k+4..k+7, for A
// and for B alike.  SwiGLU: row g is the gate row of feature f, row g+8 its up row.
// With TR = 2 a warp streams two 16-row tiles and uses its token fragments for both, which
// halves the activation traffic from L2 per weight byte.
//
// Each thread prefetches exactly the 16-byte pieces it will consume itself, STAGES k-steps
// ahead, with cp.async into a ring of its own in shared memory: the bytes in flight per
// SM are set by the ring depth, not by registers or occupancy, and no barrier is needed
// (nobody else reads a thread's slots).  WARPS is chosen from (N, K) alone -- never from
// M -- so that matrices with few row tiles (N = 4096: 256 tiles) still keep enough bytes
// in flight; TR and STAGES do not touch the arithmetic of a row, and the sums of squares a
// residual epilogue leaves for the next norm are exact integer sums (ls_common.cuh).
//
// SHARE (plain and residual projections of the wide kind, from 9 rows on; see mma_shape): the
// grid is one CTA per SM and CTA c takes the rows [c N / G, (c+1) N / G) -- equal shares to within
// one row, whatever the tile size -- as its TR tiles, the last one ragged: rows beyond the share
// copy nothing and are dropped in the epilogue.  SMs get equal shares of the memory system, so
// equal shares of the matrix keep all of them streaming to the end (256 tiles of 16 rows on 148
// SMs leave 40 SMs idle half of the time), and one CTA per SM has room for a ring that keeps
// 96 KB of weights in flight where two CTAs with two token tiles keep 64.  A row's arithmetic is
// the same in both cuts of the matrix.
template <int NT, int EPI, int TR, int WARPS, int STAGES, bool SHARE>
__global__ void __launch_bounds__(WARPS * 32) linear_mma_kernel(const LinArgs a)
{
    static_assert(!SHARE || EPI == EPI_STORE || EPI == EPI_RESIDUAL, "shares are cut in plain output rows");
    constexpr int T = WARPS * 32;
    extern __shared__ __align__(16) unsigned char ring[];
    TR_T0
    pdl_launch_dependents();
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const uint16_t *pa[TR], *pb[TR];
#pragma unroll
    for (int tr = 0; tr < TR; ++tr) {
        const int tile = blockIdx.x * TR + tr;
        if (EPI == EPI_SWIGLU) {
            int f = min(tile * 8 + g, a.N - 1);
            pa[tr] = a.w0 + (size_t)f * a.K;
            pb[tr] = a.w1 + (size_t)f * a.K;
        } else if (EPI == EPI_QKV) {
            const int tc = min(tile, (a.N >> 4) - 1);
            pa[tr] = weight_row(a, qkv_row(a, tc, g, 0));
            pb[tr] = weight_row(a, qkv_row(a, tc, g, 1));
        } else {
            pa[tr] = weight_row(a, tile * 16 + g);
            pb[tr] = weight_row(a, tile * 16 + g + 8);
        }
    }
    // SHARE: first row of the share, one past its last, and which of the thread's rows exist
    int u0 = 0, u1 = a.N;
    bool va[TR], vb[TR];
    if (SHARE) {
        u0 = (int)((long long)blockIdx.x * a.N / gridDim.x);
        u1 = (int)((long long)(blockIdx.x + 1) * a.N / gridDim.x);
#pragma unroll
        for (int tr = 0; tr < TR; ++tr) {
            const int n = u0 + tr * 16 + g;
            va[tr] = n < u1;
            vb[tr] = n + 8 < u1;
            pa[tr] = weight_row(a, n);
            pb[tr] = weight_row(a, n + 8);
        }
    }
    const uint16_t* hb[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) hb[nt] = a.h + (size_t)min(nt * 8 + g, a.M - 1) * a.K;
    // lanes whose token row does not exist copy nothing (zero fill) instead of re-reading row M-1
    bool hrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) hrow[nt] = nt * 8 + g < a.M;

    // region r (2 tr: row g, 2 tr + 1: row g+8, 2 TR + nt: tokens), stage s, thread tid -> 16 bytes
    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(ring) + (uint32_t)tid * 16u;
    auto slot = [&](int r, int s) { return ring0 + (uint32_t)((r * STAGES + s) * T) * 16u; };

    const int nsteps = (a.K + 31) >> 5;
    auto issue_w = [&](int step, int s) {  // weights: immutable, may be fetched before pdl_wait()
        if (step < nsteps) {
            const int k = step * 32 + 8 * t;
            const int nb = (k < a.K) ? 16 : 0;
            const int kk = (k < a.K) ? k : 0;
#pragma unroll
            for (int tr = 0; tr < TR; ++tr) {
                cp_async16_cg(slot(2 * tr, s), pa[tr] + kk, SHARE ? (va[tr] ? nb : 0) : nb);
                cp_async16_cg(slot(2 * tr + 1, s), pb[tr] + kk, SHARE ? (vb[tr] ? nb : 0) : nb);
            }
        }
    };
    auto issue_h = [&](int step, int s) {  // activations: written by the previous kernel
        if (step < nsteps) {
            const int k = step * 32 + 8 * t;
            const int nb = (k < a.K) ? 16 : 0;
            const int kk = (k < a.K) ? k : 0;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) cp_async16_ca(slot(2 * TR + nt, s), hb[nt] + kk, hrow[nt] ? nb : 0);
        }
    };

    float c[TR][NT][4];
#pragma unroll
    for (int tr = 0; tr < TR; ++tr)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) c[tr][nt][i] = 0.f;

    // the first STAGES-1 steps of weights are on their way while the predecessor finishes --
    // unless this is a draft pass and the step's stop mark, read past L1, already says that
    // drafting ended before it (the binding decision is the one after the wait)
    bool early = true;
    if (a.gate > 0 && a.ctl) early = a.gate <= __ldcg(a.ctl + CTL_D_EFF);
    if (early) {
#pragma unroll
        for (int p = 0; p < STAGES - 1; ++p) issue_w(warp + p * WARPS, p);
    }
    pdl_wait();
    TR_T1
    if (pass_idle(a.ctl, a.gate)) {
        cp_async_commit();
        cp_async_wait<0>();
        return;
    }
    if (!early) {
#pragma unroll
        for (int p = 0; p < STAGES - 1; ++p) issue_w(warp + p * WARPS, p);
    }
#pragma unroll
    for (int p = 0; p < STAGES - 1; ++p) {
        issue_h(warp + p * WARPS, p);
        cp_async_commit();
    }
    __shared__ float rs[kMaxRows];
    if (a.ss_in && tid < 256)  // fused RMSNorm: per-row scales, fetched while the first stages travel
        rms_rscales(a.ss_in, a.ss_clear, a.M, a.inv_d, a.eps, rs);
    // what the epilogue will need from global memory is fetched now, while the ring fills:
    // the residual values and gains (EPI_RESIDUAL), the rotation factors (EPI_QKV)
    constexpr int FRAGS = TR * NT;
    float xin[4] = {0.f, 0.f, 0.f, 0.f}, gA[2] = {0.f, 0.f}, gB[2] = {0.f, 0.f}, rsn[2] = {0.f, 0.f}, rcs[2] = {1.f, 1.f};
    int pos_epi[2] = {0, 0};  // positions of the thread's two token rows (EPI_QKV)
    if (tid < 32 * FRAGS) {
        const int efr = tid >> 5, etile = blockIdx.x * TR + efr / NT, em0 = (efr % NT) * 8 + 2 * t;
        if (EPI == EPI_RESIDUAL) {
            const int nlo = SHARE ? u0 + (efr / NT) * 16 + g : etile * 16 + g, nhi = nlo + 8;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = em0 + (i & 1), n = (i < 2) ? nlo : nhi;
                if (m < a.M && n < u1) xin[i] = a.out[(size_t)m * a.ldo + n];
            }
            if (nlo < u1) {
                if (a.hout_a) gA[0] = bf16f(a.gain_a[nlo]);
                if (a.hout_b) gB[0] = bf16f(a.gain_b[nlo]);
            }
            if (nhi < u1) {
                if (a.hout_a) gA[1] = bf16f(a.gain_a[nhi]);
                if (a.hout_b) gB[1] = bf16f(a.gain_b[nhi]);
            }
        } else if (EPI == EPI_QKV) {
            pos_epi[0] = row_pos(a, min(em0, a.M - 1));
            pos_epi[1] = row_pos(a, min(em0 + 1, a.M - 1));
            const int tph = a.hd >> 4;
            if (etile < (a.N >> 4) && etile / tph < a.Hq + a.Hkv) {
                const int j = (etile % tph) * 8 + g;
                qkv_rotation(a, j, pos_epi[0], rsn[0], rcs[0]);
                qkv_rotation(a, j, pos_epi[1], rsn[1], rcs[1]);
            }
        }
    }
    int rd = 0, wr = STAGES - 1;
    for (int step = warp; step < nsteps; step += WARPS) {
        issue_w(step + (STAGES - 1) * WARPS, wr);
        issue_h(step + (STAGES - 1) * WARPS, wr);
        cp_async_commit();
        cp_async_wait<STAGES - 1>();
        uint4 B[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) B[nt] = lds16(slot(2 * TR + nt, rd));
#pragma unroll
        for (int tr = 0; tr < TR; ++tr) {
            const uint4 A0 = lds16(slot(2 * tr, rd)), A1 = lds16(slot(2 * tr + 1, rd));
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                mma_bf16_16816(c[tr][nt], A0.x, A1.x, A0.y, A1.y, B[nt].x, B[nt].y);
                mma_bf16_16816(c[tr][nt], A0.z, A1.z, A0.w, A1.w, B[nt].z, B[nt].w);
            }
        }
        rd = (rd + 1 == STAGES) ? 0 : rd + 1;
        wr = (wr + 1 == STAGES) ? 0 : wr + 1;
    }
    cp_async_wait<0>();

    // cross-warp reduction in warp order (fixed), then the epilogue on 32*TR*NT threads; the
    // ring is free by now (every thread has consumed its own slots) and is reused
    __syncthreads();
    constexpr int FR = TR * NT;  // accumulator fragments per warp
    float(*red)[FR * 4][32] = reinterpret_cast<float(*)[FR * 4][32]>(ring);
    static_assert(sizeof(float) * WARPS * FR * 4 * 32 <= mma_ring_bytes<NT, TR, WARPS, STAGES>(), "ring too small");
    static_assert(32 * FR <= T, "not enough threads for the epilogue");
#pragma unroll
    for (int tr = 0; tr < TR; ++tr)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) red[warp][(tr * NT + nt) * 4 + i][lane] = c[tr][nt][i];
    __syncthreads();
    __shared__ float vals[16 * TR][NT * 8 + 1];
    if (threadIdx.x < 32 * FR) {
        const int fr = threadIdx.x >> 5, tr = fr / NT, nt = fr % NT;
        const int tile = blockIdx.x * TR + tr;
        const int gg = lane >> 2, tt = lane & 3;
        float r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < WARPS; ++w) s += red[w][fr * 4 + i][lane];
            r[i] = s;
        }
        const int m0 = nt * 8 + 2 * tt;  // tokens m0, m0+1
        if (a.ss_in) {
            const float s0 = rs[min(m0, a.M - 1)], s1 = rs[min(m0 + 1, a.M - 1)];
            r[0] *= s0;
            r[1] *= s1;
            r[2] *= s0;
            r[3] *= s1;
        }
        if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
            const int nlo = SHARE ? u0 + tr * 16 + gg : tile * 16 + gg, nhi = nlo + 8;
            long long q[2] = {0, 0};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int m = m0 + (i & 1), n = (i < 2) ? nlo : nhi;
                if (m < a.M && n < u1) {
                    const float xn = (EPI == EPI_RESIDUAL) ? (xin[i] + r[i]) : r[i];
                    a.out[(size_t)m * a.ldo + n] = xn;
                    if (EPI == EPI_RESIDUAL) {
                        q[i & 1] += sq_fixed(xn);
                        if (a.hout_a) a.hout_a[(size_t)m * a.N + n] = f2bf(xn * gA[i >> 1]);
                        if (a.hout_b) a.hout_b[(size_t)m * a.N + n] = f2bf(xn * gB[i >> 1]);
                    }
                }
            }
            if (EPI == EPI_RESIDUAL && a.ss_out) {  // sum over the tile's 16 rows: lanes of equal tt
#pragma unroll
                for (int sh = 4; sh < 32; sh <<= 1) {
                    q[0] += __shfl_xor_sync(0xffffffffu, q[0], sh);
                    q[1] += __shfl_xor_sync(0xffffffffu, q[1], sh);
                }
                if (gg == 0) {
                    if (m0 < a.M) ss_add(a.ss_out + (size_t)m0 * kSsSlots, q[0]);
                    if (m0 + 1 < a.M) ss_add(a.ss_out + (size_t)(m0 + 1) * kSsSlots, q[1]);
                }
            }
        } else if (EPI == EPI_SWIGLU) {
            const int f = tile * 8 + gg;
            if (f < a.N) {
                if (m0 < a.M) a.out_bf16[(size_t)m0 * a.N + f] = f2bf(silu_mul(r[0], r[2]));
                if (m0 + 1 < a.M) a.out_bf16[(size_t)(m0 + 1) * a.N + f] = f2bf(silu_mul(r[1], r[3]));
            }
        } else if (EPI == EPI_QKV) {
            if (tile < (a.N >> 4)) {
                const int tph = a.hd >> 4;
                const int head = tile / tph, j = (tile % tph) * 8 + gg;
                if (m0 < a.M) qkv_store(a, head, j, m0, pos_epi[0], r[0], r[2], rsn[0], rcs[0]);
                if (m0 + 1 < a.M) qkv_store(a, head, j, m0 + 1, pos_epi[1], r[1], r[3], rsn[1], rcs[1]);
            }
        } else {
            vals[tr * 16 + gg][m0] = r[0];
            vals[tr * 16 + gg][m0 + 1] = r[1];
            vals[tr * 16 + gg + 8][m0] = r[2];
            vals[tr * 16 + gg + 8][m0 + 1] = r[3];
        }
    }
    if (EPI == EPI_ARGMAX) {
        __syncthreads();
        if (threadIdx.x < a.M) {
            const int m = threadIdx.x;
            float v = -INFINITY, s2 = -INFINITY;
            int idx = 0x7fffffff;
#pragma unroll
            for (int rr = 0; rr < 16 * TR; ++rr) {
                int n = blockIdx.x * 16 * TR + rr;
                if (n < a.N) {
                    float x = vals[rr][m];
                    if (a.out) a.out[(size_t)m * a.ldo + n] = x;
                    top2_push(x, n, v, idx, s2);
                }
            }
            ValIdx e;
            e.v = v;
            e.i = idx;
            a.cand[(size_t)m * a.cand_stride + blockIdx.x] = e;
            if (a.second) a.second[(size_t)m * a.cand_stride + blockIdx.x] = s2;
        }
    }
    TR_END(a.w0, a.M > 1 ? 1 : 0)
}

// =============================================================================== launchers
inline int lin_grid(int epi, int N) { return epi == EPI_SWIGLU ? (N + 7) / 8 : (N + 15) / 16; }

template <int EPI>
inline cudaError_t launch_linear_fma(const LinArgs& a, const LaunchCtx& lc)
{
    dim3 grid(lin_grid(EPI, a.N)), block(128);
    if (a.M <= 1) return launch(lc, linear_fma_kernel<1, EPI>, grid, block, 0, a);
    if (a.M <= 2) return launch(lc, linear_fma_kernel<2, EPI>, grid, block, 0, a);
    if (a.M <= 4) return launch(lc, linear_fma_kernel<4, EPI>, grid, block, 0, a);
    if (a.M <= 8) return launch(lc, linear_fma_kernel<8, EPI>, grid, block, 0, a);
    return launch(lc, linear_fma_kernel<16, EPI>, grid, block, 0, a);
}

// SMs of the current device (a wide matrix from 9 rows on is cut into one share per SM)
inline int device_sms()
{
    static int sms[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!sms[dev] && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms[dev] = 0;
    return sms[dev];
}

// A row's bits depend on how K is split over the warps of its tile, and on nothing else (the
// sums of squares for the next norm are exact).  So the warps per tile come from the matrix
// shape alone (never from M):
//   few row tiles (under 350: N = 4096, 5120) -> 16 warps, 4 stages (3 with two token tiles),
//                                2 CTAs per SM, (about) one wave.  (The 384 tiles of the Llama-3-8B
//                                q|k|v are better off with 8 warps, 3 CTAs per SM and one full wave:
//                                alone 11.6 -> 14.9 us, but inside the loop the pass is 3 % faster.)
//   otherwise                 -> 8 warps, 6 stages (4 with two token tiles), 3 CTAs per SM
// while everything else may follow the pass size.  From 6 rows on, where the token rows are
// a third or more of what a tile pulls through L1, a CTA of a matrix with 700 or more row
// tiles (q|k|v, gate-up, LM head on the 7B shape) takes two tiles with 3 stages (still 3 CTAs
// per SM) and uses its token fragments for both.  Measured on the 7B shape: gate-up 32.5 ->
// 31.6 us and q|k|v 20.8 -> 19.4 us at 7 rows, 36.4 -> 33.3 us and 22.5 -> 20.2 us at 9 rows;
// below 6 rows the single tile with the deeper ring is faster -- except for q|k|v, which takes two
// tiles at every pass size: its CTAs then fit the device in one wave (384 on the 7B shape), they
// all end together, and the attention clusters that follow on the stream are placed at once
// instead of trickling in behind a second wave (in the loop: q|k|v 19.5 -> 17.9 us at 1 row).
// From 9 rows on (two token tiles, whose fragments take ring space) the plain and residual
// projections of the 16-warp kind are cut into one share of rows per SM (SHARE in
// linear_mma_kernel), 2 or 3 tiles per CTA with 4 or 3 stages: 13B shape at 9 rows, down-proj
// 35.2 -> 27.6 us and o-proj 15.6 -> 12.9 us; 7B shape, 21.1 -> 18.9 and 10.3 -> 9.9 us.
inline bool mma_wide(int epi, int N, int K)
{
    const int tiles = lin_grid(epi, N), nsteps = (K + 31) / 32;
    return tiles < 350 && nsteps >= 16;
}
inline bool mma_pair(int epi, int N, int K, int M)
{
    return (M >= 6 || epi == EPI_QKV) && !mma_wide(epi, N, K) && lin_grid(epi, N) >= 700;
}
// tiles per CTA of the one-share-per-SM cut, or 0 where it does not apply
inline int mma_share_tiles(int epi, int N, int K, int M)
{
    if ((epi != EPI_STORE && epi != EPI_RESIDUAL) || M <= 8 || !mma_wide(epi, N, K)) return 0;
    const int sms = device_sms();
    if (sms < 1 || sms >= lin_grid(epi, N)) return 0;
    const int per_sm = ((N + sms - 1) / sms + 15) / 16;
    return (per_sm == 2 || per_sm == 3) ? per_sm : 0;
}
// CTAs the MMA family launches for this matrix (also the number of argmax candidates per row)
inline int mma_grid(int epi, int N, int K, int M)
{
    const int tiles = lin_grid(epi, N);
    return mma_pair(epi, N, K, M) ? (tiles + 1) / 2 : tiles;
}

template <int NT, int EPI, int TR, int WARPS, int STAGES, bool SHARE = false>
inline cudaError_t launch_linear_mma_cfg(const LinArgs& a, const LaunchCtx& lc)
{
    constexpr size_t smem = mma_ring_bytes<NT, TR, WARPS, STAGES>();
    static bool allowed[64] = {false};  // per instantiation and device: the attribute is set once
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !allowed[dev]) {
        e = cudaFuncSetAttribute(linear_mma_kernel<NT, EPI, TR, WARPS, STAGES, SHARE>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) allowed[dev] = true;
    }
    const int tiles = lin_grid(EPI, a.N);
    return launch(lc, linear_mma_kernel<NT, EPI, TR, WARPS, STAGES, SHARE>, dim3(SHARE ? device_sms() : (tiles + TR - 1) / TR),
                  dim3(WARPS * 32), smem, a);
}

template <int EPI, bool PLAIN = (EPI == EPI_STORE || EPI == EPI_RESIDUAL)>
struct MmaShareLaunch {
    static cudaError_t run(const LinArgs&, const LaunchCtx&, int) { return cudaErrorInvalidValue; }
};
template <int EPI>
struct MmaShareLaunch<EPI, true> {
    static cudaError_t run(const LinArgs& a, const LaunchCtx& lc, int tr)
    {
        return tr == 2 ? launch_linear_mma_cfg<2, EPI, 2, 16, 4, true>(a, lc) : launch_linear_mma_cfg<2, EPI, 3, 16, 3, true>(a, lc);
    }
};

template <int EPI>
inline cudaError_t launch_linear_mma(const LinArgs& a, const LaunchCtx& lc)
{
    if (const int tr = mma_share_tiles(EPI, a.N, a.K, a.M)) return MmaShareLaunch<EPI>::run(a, lc, tr);
    if (mma_wide(EPI, a.N, a.K))
        return a.M <= 8 ? launch_linear_mma_cfg<1, EPI, 1, 16, 4>(a, lc) : launch_linear_mma_cfg<2, EPI, 1, 16, 3>(a, lc);
    if (mma_pair(EPI, a.N, a.K, a.M))
        return a.M <= 8 ? launch_linear_mma_cfg<1, EPI, 2, 8, 3>(a, lc) : launch_linear_mma_cfg<2, EPI, 2, 8, 3>(a, lc);
    if (a.M <= 8) return launch_linear_mma_cfg<1, EPI, 1, 8, 6>(a, lc);
    return launch_linear_mma_cfg<2, EPI, 1, 8, 4>(a, lc);
}

// path: 1 = FMA, 2 = MMA
inline cudaError_t launch_linear(int path, int epi, const LinArgs& a, const LaunchCtx& st)
{
    if (path == 1) {
        switch (epi) {
            case EPI_STORE: return launch_linear_fma<EPI_STORE>(a, st);
            case EPI_RESIDUAL: return launch_linear_fma<EPI_RESIDUAL>(a, st);
            case EPI_SWIGLU: return launch_linear_fma<EPI_SWIGLU>(a, st);
            case EPI_QKV: return launch_linear_fma<EPI_QKV>(a, st);
            default: return launch_linear_fma<EPI_ARGMAX>(a, st);
        }
    }
    switch (epi) {
        case EPI_STORE: return launch_linear_mma<EPI_STORE>(a, st);
        case EPI_RESIDUAL: return launch_linear_mma<EPI_RESIDUAL>(a, st);
        case EPI_SWIGLU: return launch_linear_mma<EPI_SWIGLU>(a, st);
        case EPI_QKV: return launch_linear_mma<EPI_QKV>(a, st);
        default: return launch_linear_mma<EPI_ARGMAX>(a, st);
    }
}

}  // namespace ls

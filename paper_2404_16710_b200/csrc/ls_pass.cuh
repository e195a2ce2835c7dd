// One pass of the decode loop as ONE resident kernel.
//
// A pass is what the loop of LayerSkip's self-speculative decoding (Sec. 4.3, Appendix A.4)
// does between two points where a token is known: a draft pass (embedding, layers 0..E-1, the
// shared head, argmax), the extra early pass, or the verify pass (layers E..L-1 on d+1 rows,
// head, argmax, match + crop).  At batch 1 every step of a pass is bound by the weight bytes
// it streams, and every step needs the whole output of the step before it, so a pass run as
// one kernel per step pays a launch boundary (drain, launch, refill) fifteen to forty times
// per layer-millisecond.  Here the whole pass is one cooperative kernel of as many CTAs as
// fit on the GPU; the steps are separated by a grid-wide barrier, and before a CTA waits at a
// barrier it has already issued the weight loads of its next tile, so HBM keeps streaming
// through the barrier.
//
// The arithmetic of a tile is that of linear_mma_kernel with 8 warps per tile for every
// matrix: a row's bits depend on the split of K over the warps of its tile and on nothing
// else -- not on the pass size, not on which CTA runs the tile -- so verification stays
// bit-identical to single-token decoding.
//
// The kernel stays resident while other CTAs produce its inputs, so nothing that is written
// during the pass is ever read through L1 (cp.async.cg, ld.global.cg).  Every wait is
// bounded: a barrier that does not complete within about a second records
// DEV_BARRIER_TIMEOUT in the status word and the CTA returns.
#pragma once
#include "ls_linear.cuh"

namespace ls {

constexpr int kPassThreads = 256, kPassWarps = 8;

struct PassLayer {
    const uint16_t *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *wg, *wu, *wd;
};

struct PassModel {  // fixed for a model
    const PassLayer* layers;  // device array [L]
    const uint16_t *emb, *fnorm, *lm;
    int D, Hq, Hkv, hd, F, V, page_shift, max_seq, n_part, chunk_cap, cand_stride;
    float eps, theta;
    const float* inv_freq;
    const int32_t* page_table;
    uint16_t *kpages, *vpages;
    size_t layer_kv_elems;
    float *x, *ss, *part;
    uint16_t *h, *hE, *q, *o, *a;
    int32_t *attn_counters, *ctl, *draft, *verified, *out_ids, *accepted, *drafted;
    ValIdx* cand;
    float* second;
    unsigned* bar;  // [0] arrivals, [1] generation, [2] rows whose argmax is finished
};

struct PassArgs {  // one launch
    int l0, l1, M, slot, pos_off, gate;
    const int32_t* tok;          // ids to embed into the rows first, or nullptr (rows hold x already)
    const uint16_t* h_first;     // x*gain rows feeding layer l0 (unused when tok != nullptr)
    const uint16_t* gain_end_a;  // after the last layer: x*gain_end_a -> the h rows (nullptr: none)
    const uint16_t* gain_end_b;  //                       x*gain_end_b -> the exit-activation rows
    int head;                    // shared head + argmax after the layers
    int32_t* tok_out;
    float* logits;               // optional fp32 [M][V]
    float min_margin;            // > 0: adaptive drafting, this is the head of draft pass `gate`
    int accept_d;                // >= 0: match + crop with this many drafts after the head
    int adaptive;
};

template <int NT>
struct PassCfg {
    static constexpr int kStages = NT == 1 ? 5 : 4;
    static constexpr int kRingBytes = (2 + NT) * kStages * kPassThreads * 16;
    static constexpr int kRedBytes = kPassWarps * NT * 4 * 32 * 4;
    static constexpr int kLinBytes = kRingBytes + kRedBytes;
};

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier over a co-resident grid (cooperative launch).  gen is the generation the
// CTA expects to leave behind.  false: the barrier did not complete in time.
__device__ __forceinline__ bool grid_sync(unsigned* bar, unsigned& gen, int32_t* ctl)
{
    __shared__ int ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        ok = 1;
        __threadfence();
        const unsigned prev = atomicAdd(bar, 1u);
        if (prev == gridDim.x - 1) {
            atomicExch(bar, 0u);
            __threadfence();
            atomicExch(bar + 1, gen + 1);
        } else {
            unsigned it = 0;
            while (ld_acquire_u32(bar + 1) == gen) {
                if (++it > 4096u) {
                    __nanosleep(500);
                    if (it > 4096u + (1u << 21)) {  // about a second
                        ok = 0;
                        atomicExch(reinterpret_cast<unsigned*>(ctl + CTL_STATUS), (unsigned)DEV_BARRIER_TIMEOUT);
                        break;
                    }
                }
            }
        }
        __threadfence();
    }
    __syncthreads();
    ++gen;
    return ok != 0;
}

// ------------------------------------------------------------------ one 16-row weight tile
template <int EPI>
__device__ __forceinline__ void tile_rows(const LinArgs& a, int tile, const uint16_t*& pa, const uint16_t*& pb)
{
    const int g = (threadIdx.x & 31) >> 2;
    if (EPI == EPI_SWIGLU) {
        const int f = min(tile * 8 + g, a.N - 1);
        pa = a.w0 + (size_t)f * a.K;
        pb = a.w1 + (size_t)f * a.K;
    } else if (EPI == EPI_QKV) {
        const int tc = min(tile, (a.N >> 4) - 1);
        pa = weight_row(a, qkv_row(a, tc, g, 0));
        pb = weight_row(a, qkv_row(a, tc, g, 1));
    } else {
        pa = weight_row(a, tile * 16 + g);
        pb = weight_row(a, tile * 16 + g + 8);
    }
}

template <int NT>
__device__ __forceinline__ uint32_t ring_slot(uint32_t ring0, int r, int s)
{
    return ring0 + (uint32_t)((r * PassCfg<NT>::kStages + s) * kPassThreads) * 16u;
}

// the thread's weight pieces of its first STAGES-1 k-steps (weights never change: this may
// run long before the tile's inputs exist)
template <int NT, int EPI>
__device__ __forceinline__ void tile_prefetch(const LinArgs& a, int tile, uint32_t ring0)
{
    constexpr int STAGES = PassCfg<NT>::kStages;
    const int warp = threadIdx.x >> 5, t = threadIdx.x & 3;
    const uint16_t *pa, *pb;
    tile_rows<EPI>(a, tile, pa, pb);
    const int nsteps = (a.K + 31) >> 5;
#pragma unroll
    for (int p = 0; p < STAGES - 1; ++p) {
        const int step = warp + p * kPassWarps;
        if (step < nsteps) {
            const int k = step * 32 + 8 * t;
            const int nb = (k < a.K) ? 16 : 0;
            const int kk = (k < a.K) ? k : 0;
            cp_async16_cg(ring_slot<NT>(ring0, 0, p), pa + kk, nb);
            cp_async16_cg(ring_slot<NT>(ring0, 1, p), pb + kk, nb);
        }
    }
}

// The tile itself; tile_prefetch(a, tile) has been issued by this CTA and nothing else has
// touched the ring since.  after_k() runs when the thread has consumed its ring (the place
// to prefetch the next tile), before the cross-warp reduction and the epilogue.
template <int NT, int EPI, class AfterK>
__device__ __forceinline__ void tile_run(const LinArgs& a, int tile, uint32_t ring0, float* red_raw, float* rs,
                                         float (*vals)[NT * 8 + 1], AfterK after_k)
{
    constexpr int STAGES = PassCfg<NT>::kStages, WARPS = kPassWarps;
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const uint16_t *pa, *pb;
    tile_rows<EPI>(a, tile, pa, pb);
    const uint16_t* hb[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) hb[nt] = a.h + (size_t)min(nt * 8 + g, a.M - 1) * a.K;
    const int nsteps = (a.K + 31) >> 5;
    auto issue_w = [&](int step, int s) {
        if (step < nsteps) {
            const int k = step * 32 + 8 * t;
            const int nb = (k < a.K) ? 16 : 0;
            const int kk = (k < a.K) ? k : 0;
            cp_async16_cg(ring_slot<NT>(ring0, 0, s), pa + kk, nb);
            cp_async16_cg(ring_slot<NT>(ring0, 1, s), pb + kk, nb);
        }
    };
    auto issue_h = [&](int step, int s) {
        if (step < nsteps) {
            const int k = step * 32 + 8 * t;
            const int nb = (k < a.K) ? 16 : 0;
            const int kk = (k < a.K) ? k : 0;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) cp_async16_cg(ring_slot<NT>(ring0, 2 + nt, s), hb[nt] + kk, nb);
        }
    };
    float c[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) c[nt][i] = 0.f;

    __syncthreads();  // the previous tile's epilogue is done with rs and vals
#pragma unroll
    for (int p = 0; p < STAGES - 1; ++p) {
        issue_h(warp + p * WARPS, p);
        cp_async_commit();
    }
    if (a.ss_in) {
        for (int m = warp; m < a.M; m += WARPS) {
            const float v = row_rscale(a, m, lane);
            if (lane == 0) rs[m] = v;
        }
    }
    // what the epilogue needs from global memory, fetched while the ring fills
    float xin[4] = {0.f, 0.f, 0.f, 0.f}, gA[2] = {0.f, 0.f}, gB[2] = {0.f, 0.f}, rsn[2] = {0.f, 0.f}, rcs[2] = {1.f, 1.f};
    if (tid < 32 * NT) {
        const int em0 = (tid >> 5) * 8 + 2 * t;
        if (EPI == EPI_RESIDUAL) {
            const int nlo = tile * 16 + g, nhi = nlo + 8;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = em0 + (i & 1), n = (i < 2) ? nlo : nhi;
                if (m < a.M && n < a.N) xin[i] = __ldcg(a.out + (size_t)m * a.ldo + n);
            }
            if (nlo < a.N) {
                if (a.hout_a) gA[0] = bf16f(a.gain_a[nlo]);
                if (a.hout_b) gB[0] = bf16f(a.gain_b[nlo]);
            }
            if (nhi < a.N) {
                if (a.hout_a) gA[1] = bf16f(a.gain_a[nhi]);
                if (a.hout_b) gB[1] = bf16f(a.gain_b[nhi]);
            }
        } else if (EPI == EPI_QKV) {
            const int tph = a.hd >> 4;
            if (tile < (a.N >> 4) && tile / tph < a.Hq + a.Hkv) {
                const int j = (tile % tph) * 8 + g;
                qkv_rotation(a, j, a.pos_off + em0, rsn[0], rcs[0]);
                qkv_rotation(a, j, a.pos_off + em0 + 1, rsn[1], rcs[1]);
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
        for (int nt = 0; nt < NT; ++nt) B[nt] = lds16(ring_slot<NT>(ring0, 2 + nt, rd));
        const uint4 A0 = lds16(ring_slot<NT>(ring0, 0, rd)), A1 = lds16(ring_slot<NT>(ring0, 1, rd));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            mma_bf16_16816(c[nt], A0.x, A1.x, A0.y, A1.y, B[nt].x, B[nt].y);
            mma_bf16_16816(c[nt], A0.z, A1.z, A0.w, A1.w, B[nt].z, B[nt].w);
        }
        rd = (rd + 1 == STAGES) ? 0 : rd + 1;
        wr = (wr + 1 == STAGES) ? 0 : wr + 1;
    }
    cp_async_wait<0>();
    after_k();

    // cross-warp reduction in warp order (fixed), then the epilogue on 32*NT threads
    float(*red)[NT * 4][32] = reinterpret_cast<float(*)[NT * 4][32]>(red_raw);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) red[warp][nt * 4 + i][lane] = c[nt][i];
    __syncthreads();
    if (tid < 32 * NT) {
        const int nt = tid >> 5;
        float r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < WARPS; ++w) s += red[w][nt * 4 + i][lane];
            r[i] = s;
        }
        const int m0 = nt * 8 + 2 * t;  // tokens m0, m0+1
        if (a.ss_in) {
            const float s0 = rs[min(m0, a.M - 1)], s1 = rs[min(m0 + 1, a.M - 1)];
            r[0] *= s0;
            r[1] *= s1;
            r[2] *= s0;
            r[3] *= s1;
        }
        if (EPI == EPI_STORE || EPI == EPI_RESIDUAL) {
            const int nlo = tile * 16 + g, nhi = nlo + 8;
            float q[2] = {0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = m0 + (i & 1), n = (i < 2) ? nlo : nhi;
                if (m < a.M && n < a.N) {
                    const float xn = (EPI == EPI_RESIDUAL) ? (xin[i] + r[i]) : r[i];
                    a.out[(size_t)m * a.ldo + n] = xn;
                    if (EPI == EPI_RESIDUAL) {
                        q[i & 1] = fmaf(xn, xn, q[i & 1]);
                        if (a.hout_a) a.hout_a[(size_t)m * a.N + n] = f2bf(xn * gA[i >> 1]);
                        if (a.hout_b) a.hout_b[(size_t)m * a.N + n] = f2bf(xn * gB[i >> 1]);
                    }
                }
            }
            if (EPI == EPI_RESIDUAL && a.ss_out) {
#pragma unroll
                for (int sh = 4; sh < 32; sh <<= 1) {
                    q[0] += __shfl_xor_sync(0xffffffffu, q[0], sh);
                    q[1] += __shfl_xor_sync(0xffffffffu, q[1], sh);
                }
                if (g == 0) {
                    if (m0 < a.M) a.ss_out[(size_t)m0 * a.ss_stride + tile] = q[0];
                    if (m0 + 1 < a.M) a.ss_out[(size_t)(m0 + 1) * a.ss_stride + tile] = q[1];
                }
            }
        } else if (EPI == EPI_SWIGLU) {
            const int f = tile * 8 + g;
            if (f < a.N) {
                if (m0 < a.M) a.out_bf16[(size_t)m0 * a.N + f] = f2bf(silu_mul(r[0], r[2]));
                if (m0 + 1 < a.M) a.out_bf16[(size_t)(m0 + 1) * a.N + f] = f2bf(silu_mul(r[1], r[3]));
            }
        } else if (EPI == EPI_QKV) {
            if (tile < (a.N >> 4)) {
                const int tph = a.hd >> 4;
                const int head = tile / tph, j = (tile % tph) * 8 + g;
                if (m0 < a.M) qkv_store(a, head, j, m0, a.pos_off, r[0], r[2], rsn[0], rcs[0]);
                if (m0 + 1 < a.M) qkv_store(a, head, j, m0 + 1, a.pos_off, r[1], r[3], rsn[1], rcs[1]);
            }
        } else {
            vals[g][m0] = r[0];
            vals[g][m0 + 1] = r[1];
            vals[g + 8][m0] = r[2];
            vals[g + 8][m0 + 1] = r[3];
        }
    }
    if (EPI == EPI_ARGMAX) {
        __syncthreads();
        if (tid < a.M) {
            const int m = tid;
            float v = -INFINITY, s2 = -INFINITY;
            int idx = 0x7fffffff;
#pragma unroll
            for (int rr = 0; rr < 16; ++rr) {
                const int n = tile * 16 + rr;
                if (n < a.N) {
                    const float x = vals[rr][m];
                    if (a.out) a.out[(size_t)m * a.ldo + n] = x;
                    top2_push(x, n, v, idx, s2);
                }
            }
            ValIdx e;
            e.v = v;
            e.i = idx;
            a.cand[(size_t)m * a.cand_stride + tile] = e;
            if (a.second) a.second[(size_t)m * a.cand_stride + tile] = s2;
        }
    }
}

// ------------------------------------------------------------------ the steps of a pass
enum PassStep : int { PS_QKV = 0, PS_ATT = 1, PS_O = 2, PS_GU = 3, PS_DOWN = 4, PS_PER_LAYER = 5 };

// step s of the pass: layer l0 + s / 5, kind s % 5; s == 5 (l1 - l0) is the head
struct PassView {
    const PassModel& pm;
    const PassArgs& pa;
    int pos0;
    __device__ __forceinline__ int n_steps() const { return (pa.l1 - pa.l0) * PS_PER_LAYER + (pa.head ? 1 : 0); }
    __device__ __forceinline__ int kind(int s) const
    {
        return s >= (pa.l1 - pa.l0) * PS_PER_LAYER ? (int)PS_PER_LAYER : s % PS_PER_LAYER;
    }
    __device__ __forceinline__ int tiles(int s) const
    {
        switch (kind(s)) {
            case PS_QKV: return ((pm.Hq + 2 * pm.Hkv) * pm.hd) >> 4;
            case PS_ATT: return 0;
            case PS_O: return (pm.D + 15) >> 4;
            case PS_GU: return (pm.F + 7) >> 3;
            case PS_DOWN: return (pm.D + 15) >> 4;
            default: return (pm.V + 15) >> 4;
        }
    }
    __device__ __forceinline__ LinArgs lin(int s) const
    {
        LinArgs a;
        memset(&a, 0, sizeof(a));
        const int k = kind(s);
        const int l = pa.l0 + s / PS_PER_LAYER;
        const int D = pm.D, qw = pm.Hq * pm.hd, kvw = pm.Hkv * pm.hd;
        uint16_t* hrow = pm.h + (size_t)pa.slot * D;
        float* xrow = pm.x + (size_t)pa.slot * D;
        a.M = pa.M;
        a.ss_stride = pm.n_part;
        a.n_part = pm.n_part;
        a.inv_d = 1.0f / (float)D;
        a.eps = pm.eps;
        if (k == PS_PER_LAYER) {  // the shared head
            a.w0 = a.w1 = a.w2 = pm.lm;
            a.n0 = a.N = pm.V;
            a.K = D;
            a.h = hrow;
            a.cand = pm.cand;
            a.cand_stride = pm.cand_stride;
            a.second = pa.min_margin > 0.f ? pm.second : nullptr;
            a.out = pa.logits;
            a.ldo = pm.V;
            a.ss_in = pm.ss + (size_t)pa.slot * pm.n_part;
            return a;
        }
        const PassLayer& w = pm.layers[l];
        if (k == PS_QKV) {
            a.w0 = w.wq;
            a.w1 = w.wk;
            a.w2 = w.wv;
            a.n0 = qw;
            a.n1 = kvw;
            a.N = qw + 2 * kvw;
            a.K = D;
            a.h = (l == pa.l0 && !pa.tok) ? pa.h_first : hrow;
            a.inv_freq = pm.inv_freq;
            a.page_table = pm.page_table;
            a.q_out = pm.q;
            a.kpages = pm.kpages + (size_t)l * pm.layer_kv_elems;
            a.vpages = pm.vpages + (size_t)l * pm.layer_kv_elems;
            a.Hq = pm.Hq;
            a.Hkv = pm.Hkv;
            a.hd = pm.hd;
            a.page_shift = pm.page_shift;
            a.max_seq = pm.max_seq;
            a.pos_off = pos0;  // absolute: a.ctl stays null
            a.theta = pm.theta;
            a.ss_in = pm.ss + (size_t)pa.slot * pm.n_part;
        } else if (k == PS_O) {
            a.w0 = a.w1 = a.w2 = w.wo;
            a.n0 = a.N = D;
            a.K = qw;
            a.h = pm.o;
            a.out = xrow;
            a.ldo = D;
            a.ss_out = pm.ss + (size_t)pa.slot * pm.n_part;
            a.gain_a = w.ffn_norm;
            a.hout_a = hrow;
        } else if (k == PS_GU) {
            a.w0 = w.wg;
            a.w1 = w.wu;
            a.w2 = w.wu;
            a.n0 = a.N = pm.F;
            a.K = D;
            a.h = hrow;
            a.out_bf16 = pm.a;
            a.ss_in = pm.ss + (size_t)pa.slot * pm.n_part;
        } else {  // PS_DOWN
            a.w0 = a.w1 = a.w2 = w.wd;
            a.n0 = a.N = D;
            a.K = pm.F;
            a.h = pm.a;
            a.out = xrow;
            a.ldo = D;
            a.ss_out = pm.ss + (size_t)pa.slot * pm.n_part;
            if (l + 1 < pa.l1) {
                a.gain_a = pm.layers[l + 1].attn_norm;
                a.hout_a = hrow;
            } else {
                a.gain_a = pa.gain_end_a;
                a.hout_a = pa.gain_end_a ? hrow : nullptr;
                a.gain_b = pa.gain_end_b;
                a.hout_b = pa.gain_end_b ? pm.hE + (size_t)pa.slot * D : nullptr;
            }
        }
        return a;
    }
};

template <int NT>
__device__ __forceinline__ void step_prefetch(const PassView& v, int s, int tile, uint32_t ring0)
{
    const LinArgs a = v.lin(s);
    switch (v.kind(s)) {
        case PS_QKV: tile_prefetch<NT, EPI_QKV>(a, tile, ring0); break;
        case PS_GU: tile_prefetch<NT, EPI_SWIGLU>(a, tile, ring0); break;
        default: tile_prefetch<NT, EPI_RESIDUAL>(a, tile, ring0); break;  // plain row tiles: O, down, head
    }
}

// The CTA's next tile after (s, tile): the next one of the same step, else its first tile of
// a later step -- but never across an attention step, whose shared memory overlays the ring.
__device__ __forceinline__ bool next_tile(const PassView& v, int s, int tile, int& ns, int& ntile)
{
    if (tile >= 0 && tile + (int)gridDim.x < v.tiles(s)) {
        ns = s;
        ntile = tile + (int)gridDim.x;
        return true;
    }
    const int n = v.n_steps();
    for (int s2 = s + 1; s2 < n; ++s2) {
        if (v.kind(s2) == PS_ATT) return false;
        if ((int)blockIdx.x < v.tiles(s2)) {
            ns = s2;
            ntile = (int)blockIdx.x;
            return true;
        }
    }
    return false;
}

template <int NT, int HD>
__global__ void __launch_bounds__(kPassThreads, 3) pass_kernel(const __grid_constant__ PassModel pm,
                                                           const __grid_constant__ PassArgs pa)
{
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ float rs[kMaxRows];
    __shared__ float vals[16][NT * 8 + 1];
    __shared__ float ered[8];
    const int tid = threadIdx.x;
    int32_t* ctl = pm.ctl;
    // idle launches and bad positions end here, for every CTA alike (nothing below has run)
    // (a recorded fault, e.g. a barrier that timed out, idles everything after it)
    if (__ldcg(ctl + CTL_DONE) || __ldcg(ctl + CTL_STATUS) || (pa.gate > 0 && pa.gate > __ldcg(ctl + CTL_D_EFF))) return;
    const int pos0 = __ldcg(ctl + CTL_CACHE_LEN) + pa.pos_off;
    const int last_pos = pos0 + pa.M - 1;
    const int n_active = last_pos / kAttnChunk + 1;
    if (pos0 < 0 || last_pos >= pm.max_seq || n_active > pm.chunk_cap) {
        if (tid == 0 && blockIdx.x == 0) ctl[CTL_STATUS] = DEV_POS_OVERFLOW;
        return;
    }
    unsigned gen = ld_acquire_u32(pm.bar + 1);
    const PassView v{pm, pa, pos0};
    const uint32_t ring0 = (uint32_t)__cvta_generic_to_shared(dyn) + (uint32_t)tid * 16u;
    float* red = reinterpret_cast<float*>(dyn + PassCfg<NT>::kRingBytes);
    const int n_steps = v.n_steps();

    // what the ring currently holds the first stages of
    int pf_s = -1, pf_t = -1;
    auto prefetch_after = [&](int s, int tile) {
        int ns, nt;
        if (next_tile(v, s, tile, ns, nt)) {
            step_prefetch<NT>(v, ns, nt, ring0);
            pf_s = ns;
            pf_t = nt;
        }
    };
    prefetch_after(-1, -1);

    if (pa.tok) {  // embedding of the pass's rows (x_0 of Sec. 4.1) and what layer l0's fused norm needs
        if ((int)blockIdx.x < pa.M) {
            const int m = blockIdx.x, D = pm.D;
            int id = pa.tok[m];
            if (id < 0 || id >= pm.V) {
                if (tid == 0) ctl[CTL_STATUS] = DEV_BAD_TOKEN;
                id = 0;
            }
            const uint4* src = reinterpret_cast<const uint4*>(pm.emb + (size_t)id * D);
            float4* dst = reinterpret_cast<float4*>(pm.x + (size_t)(pa.slot + m) * D);
            const uint16_t* gain = pm.layers[pa.l0].attn_norm;
            uint16_t* hout = pm.h + (size_t)(pa.slot + m) * D;
            float ss = 0.f;
            for (int c = tid; c < D / 8; c += kPassThreads) {
                const uint4 e = src[c];
                const float f[8] = {bf16lo(e.x), bf16hi(e.x), bf16lo(e.y), bf16hi(e.y),
                                    bf16lo(e.z), bf16hi(e.z), bf16lo(e.w), bf16hi(e.w)};
                dst[2 * c] = make_float4(f[0], f[1], f[2], f[3]);
                dst[2 * c + 1] = make_float4(f[4], f[5], f[6], f[7]);
                const uint4 gv = reinterpret_cast<const uint4*>(gain)[c];
                const float g[8] = {bf16lo(gv.x), bf16hi(gv.x), bf16lo(gv.y), bf16hi(gv.y),
                                    bf16lo(gv.z), bf16hi(gv.z), bf16lo(gv.w), bf16hi(gv.w)};
                uint4 o;
                o.x = pack_bf16(f[0] * g[0], f[1] * g[1]);
                o.y = pack_bf16(f[2] * g[2], f[3] * g[3]);
                o.z = pack_bf16(f[4] * g[4], f[5] * g[5]);
                o.w = pack_bf16(f[6] * g[6], f[7] * g[7]);
                reinterpret_cast<uint4*>(hout)[c] = o;
#pragma unroll
                for (int i = 0; i < 8; ++i) ss = fmaf(f[i], f[i], ss);
            }
            const float tot = block_sum_256(ss, ered);
            float* so = pm.ss + (size_t)(pa.slot + m) * pm.n_part;
            for (int i = tid; i < pm.n_part; i += kPassThreads) so[i] = (i == 0) ? tot : 0.f;
        }
        if (!grid_sync(pm.bar, gen, ctl)) return;
    }

    for (int s = 0; s < n_steps; ++s) {
        const int kind = v.kind(s);
        if (kind == PS_ATT) {
            const int l = pa.l0 + s / PS_PER_LAYER;
            const uint16_t* kp = pm.kpages + (size_t)l * pm.layer_kv_elems;
            const uint16_t* vp = pm.vpages + (size_t)l * pm.layer_kv_elems;
            const int items = n_active * pm.Hkv;
            for (int it = blockIdx.x; it < items; it += gridDim.x) {
                __syncthreads();  // the previous item is done with the shared memory
                attn_item<HD>(pm.q, kp, vp, pm.page_table, pos0, pa.M, pm.Hq, pm.Hkv, pm.page_shift, pm.chunk_cap,
                              pm.part, pm.attn_counters, pm.o, it % n_active, it / n_active, n_active, dyn);
            }
            __syncthreads();
            prefetch_after(s, -1);
        } else {
            const LinArgs a = v.lin(s);
            const int nt = v.tiles(s);
            for (int tile = blockIdx.x; tile < nt; tile += gridDim.x) {
                if (pf_s != s || pf_t != tile) step_prefetch<NT>(v, s, tile, ring0);
                auto after = [&]() { prefetch_after(s, tile); };
                switch (kind) {
                    case PS_QKV: tile_run<NT, EPI_QKV>(a, tile, ring0, red, rs, vals, after); break;
                    case PS_O:
                    case PS_DOWN: tile_run<NT, EPI_RESIDUAL>(a, tile, ring0, red, rs, vals, after); break;
                    case PS_GU: tile_run<NT, EPI_SWIGLU>(a, tile, ring0, red, rs, vals, after); break;
                    default: tile_run<NT, EPI_ARGMAX>(a, tile, ring0, red, rs, vals, after); break;
                }
            }
        }
        if (!grid_sync(pm.bar, gen, ctl)) return;
    }

    if (!pa.head || (int)blockIdx.x >= pa.M) return;
    // argmax of row m over the per-tile candidates; (value desc, index asc) is a total order,
    // so the reduction tree does not matter and the lowest index wins a tie
    {
        __shared__ float sv[kPassThreads];
        __shared__ float s2[kPassThreads];
        __shared__ int si[kPassThreads];
        __shared__ int last_row;
        const int m = blockIdx.x;
        const int n_cand = (pm.V + 15) >> 4;
        const bool want2 = pa.min_margin > 0.f;
        float bv = -INFINITY, bs = -INFINITY;
        int bi = 0x7fffffff;
        for (int k = tid; k < n_cand; k += kPassThreads) {
            const size_t at = (size_t)m * pm.cand_stride + k;
            const float2 e = __ldcg(reinterpret_cast<const float2*>(pm.cand + at));
            top2_merge(e.x, __float_as_int(e.y), want2 ? __ldcg(pm.second + at) : -INFINITY, bv, bi, bs);
        }
        sv[tid] = bv;
        s2[tid] = bs;
        si[tid] = bi;
        __syncthreads();
        for (int st = kPassThreads / 2; st > 0; st >>= 1) {
            if (tid < st) {
                top2_merge(sv[tid + st], si[tid + st], s2[tid + st], bv, bi, bs);
                sv[tid] = bv;
                s2[tid] = bs;
                si[tid] = bi;
            }
            __syncthreads();
        }
        if (tid == 0) {
            pa.tok_out[m] = bi;
            if (want2 && m == 0 && bv - bs < pa.min_margin && pa.gate < ctl[CTL_D_EFF]) ctl[CTL_D_EFF] = pa.gate;
            last_row = 0;
            if (pa.accept_d >= 0) {
                __threadfence();
                const unsigned prev = atomicAdd(pm.bar + 2, 1u);
                if (prev == (unsigned)pa.M - 1) {
                    atomicExch(pm.bar + 2, 0u);
                    __threadfence();
                    last_row = 1;
                }
            }
        }
        __syncthreads();
        if (!last_row || tid != 0) return;
        // match + crop (Appendix A.4), as accept_kernel
        int d = pa.accept_d;
        if (pa.adaptive) {
            d = min(d, ctl[CTL_D_EFF]);
            ctl[CTL_D_EFF] = kNoStop;
        }
        const volatile int32_t* draft = pm.draft;
        const volatile int32_t* verified = pa.tok_out;
        int n = 0;
        while (n < d && draft[n] == verified[n]) ++n;
        int n_out = ctl[CTL_N_OUT];
        const int max_new = ctl[CTL_MAX_NEW], eos = ctl[CTL_EOS];
        bool stop = false;
        for (int i = 0; i <= n && n_out < max_new && !stop; ++i) {
            const int tk = (i < n) ? draft[i] : verified[n];
            pm.out_ids[n_out++] = tk;
            if (eos >= 0 && tk == eos) stop = true;
        }
        const int steps = ctl[CTL_N_STEPS];
        pm.accepted[steps] = n;
        if (pa.adaptive) pm.drafted[steps] = d;
        ctl[CTL_N_STEPS] = steps + 1;
        ctl[CTL_N_OUT] = n_out;
        ctl[CTL_CUR_TOK] = verified[n];
        ctl[CTL_CACHE_LEN] += n + 1;
        if (stop || n_out >= max_new) ctl[CTL_DONE] = 1;
    }
}

template <int HD>
__host__ __device__ constexpr size_t pass_smem_bytes(int NT, int group)
{
    const size_t lin = NT == 1 ? (size_t)PassCfg<1>::kLinBytes : (size_t)PassCfg<2>::kLinBytes;
    const size_t att = attn_smem_bytes<HD>(group * (NT == 1 ? 8 : 16));
    return lin > att ? lin : att;
}

}  // namespace ls

// Non-GEMV kernels of the decode loop: embedding, RMSNorm, rotary embedding + KV append,
// chunked causal attention over the paged cache with its ordered merge, argmax finish,
// accept/rollback.
//
// Invariant kept by every kernel here: the instructions that produce row m's result do
// not depend on how many rows the pass has.  The verification pass of num_draft+1 rows
// (LayerSkip Sec. 4.3.2) therefore reproduces single-token decoding bit for bit.
#pragma once
#include "ls_common.cuh"

namespace ls {

// position of row 0 of this pass: the loop's cache length plus a per-launch offset
__device__ __forceinline__ bool pass_begin(const int32_t* ctl, int pos_off, int& pos0, int gate = 0)
{
    pdl_launch_dependents();
    pdl_wait();
    if (ctl) {
        if (pass_idle(ctl, gate)) return false;
        pos0 = ctl[CTL_CACHE_LEN] + pos_off;
    } else {
        pos0 = pos_off;
    }
    return true;
}

__device__ __forceinline__ float block_sum_256(float v, float* red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red[w];
    return s;
}

// ------------------------------------------------------------------ embedding (x_0 = Emb[id])
// grid M, block 256.  tok[m] is read from device memory.  With gain != nullptr the kernel
// also leaves what the first layer's fused RMSNorm needs: hout = bf16(x * gain) and the
// row's sum of squares in ss_out[m][0] (the other n_part - 1 partial sums are zero).
__global__ void __launch_bounds__(256)
embed_kernel(const uint16_t* __restrict__ emb, const int32_t* __restrict__ tok, int D, int V,
             float* __restrict__ x, int32_t* ctl, const uint16_t* __restrict__ gain,
             uint16_t* __restrict__ hout, float* __restrict__ ss_out, int ss_stride, int n_part, int gate)
{
    __shared__ float red[8];
    pdl_launch_dependents();
    pdl_wait();
    if (pass_idle(ctl, gate)) return;
    int m = blockIdx.x;
    int id = tok[m];
    if (id < 0 || id >= V) {
        if (ctl && threadIdx.x == 0) ctl[CTL_STATUS] = DEV_BAD_TOKEN;
        id = 0;
    }
    const uint4* src = reinterpret_cast<const uint4*>(emb + (size_t)id * D);
    float4* dst = reinterpret_cast<float4*>(x + (size_t)m * D);
    float ss = 0.f;
    for (int c = threadIdx.x; c < D / 8; c += 256) {
        uint4 v = src[c];
        const float f[8] = {bf16lo(v.x), bf16hi(v.x), bf16lo(v.y), bf16hi(v.y),
                            bf16lo(v.z), bf16hi(v.z), bf16lo(v.w), bf16hi(v.w)};
        dst[2 * c] = make_float4(f[0], f[1], f[2], f[3]);
        dst[2 * c + 1] = make_float4(f[4], f[5], f[6], f[7]);
        if (gain) {
            const uint4 gv = reinterpret_cast<const uint4*>(gain)[c];
            const float g[8] = {bf16lo(gv.x), bf16hi(gv.x), bf16lo(gv.y), bf16hi(gv.y),
                                bf16lo(gv.z), bf16hi(gv.z), bf16lo(gv.w), bf16hi(gv.w)};
            uint4 o;
            o.x = pack_bf16(f[0] * g[0], f[1] * g[1]);
            o.y = pack_bf16(f[2] * g[2], f[3] * g[3]);
            o.z = pack_bf16(f[4] * g[4], f[5] * g[5]);
            o.w = pack_bf16(f[6] * g[6], f[7] * g[7]);
            reinterpret_cast<uint4*>(hout + (size_t)m * D)[c] = o;
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
        }
    }
    if (gain) {
        const float tot = block_sum_256(ss, red);
        for (int i = threadIdx.x; i < n_part; i += 256) ss_out[(size_t)m * ss_stride + i] = (i == 0) ? tot : 0.f;
    }
}

// ------------------------------------------------------------------ RMSNorm
// grid M, block 256.  out = bf16(x / sqrt(mean x^2 + eps) * g).
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const float* __restrict__ x, const uint16_t* __restrict__ g, int D, float eps,
               uint16_t* __restrict__ out, const int32_t* ctl)
{
    __shared__ float red[8];
    pdl_launch_dependents();
    pdl_wait();
    if (ctl && ctl[CTL_DONE]) return;
    int m = blockIdx.x;
    const float4* xr = reinterpret_cast<const float4*>(x + (size_t)m * D);
    float ss = 0.f;
    for (int c = threadIdx.x; c < D / 4; c += 256) {
        float4 v = xr[c];
        ss = fmaf(v.x, v.x, ss);
        ss = fmaf(v.y, v.y, ss);
        ss = fmaf(v.z, v.z, ss);
        ss = fmaf(v.w, v.w, ss);
    }
    float tot = block_sum_256(ss, red);
    float r = 1.0f / sqrtf(tot / (float)D + eps);
    const uint2* gr = reinterpret_cast<const uint2*>(g);
    uint2* o = reinterpret_cast<uint2*>(out + (size_t)m * D);
    for (int c = threadIdx.x; c < D / 4; c += 256) {
        float4 v = xr[c];
        uint2 gg = gr[c];
        uint2 w;
        w.x = pack_bf16(v.x * r * bf16lo(gg.x), v.y * r * bf16hi(gg.x));
        w.y = pack_bf16(v.z * r * bf16lo(gg.y), v.w * r * bf16hi(gg.y));
        o[c] = w;
    }
}

// ------------------------------------------------------------------ paged KV addressing
// Physical page p of a layer holds [Hkv][page_size][hd] bf16 for K (and the same for V).
__device__ __forceinline__ size_t kv_row_offset(const int32_t* __restrict__ page_table, int pos,
                                                int page_shift, int Hkv, int kh, int hd)
{
    int page = pos >> page_shift;
    int off = pos & ((1 << page_shift) - 1);
    int phys = page_table[page];
    return (((size_t)phys * Hkv + kh) * ((size_t)1 << page_shift) + off) * (size_t)hd;
}

// ------------------------------------------------------------------ RoPE + KV append
// grid (M, Hq + 2 Hkv), block hd/2.  Row m sits at position pos0 + m.  Pairs (j, j + hd/2)
// are rotated by pos * theta^(-2j/hd).  q -> bf16 [M, Hq*hd]; k, v -> bf16 cache rows.
__global__ void rope_append_kernel(const float* __restrict__ qkv, int Hq, int Hkv, int hd,
                                   const float* __restrict__ inv_freq, float theta, int page_shift,
                                   const int32_t* __restrict__ page_table, int max_seq,
                                   uint16_t* __restrict__ q_out, uint16_t* __restrict__ kpages,
                                   uint16_t* __restrict__ vpages, int32_t* ctl, int pos_off)
{
    int pos0;
    if (!pass_begin(ctl, pos_off, pos0)) return;
    int m = blockIdx.x, h = blockIdx.y, j = threadIdx.x, half = hd >> 1;
    int pos = pos0 + m;
    if (pos < 0 || pos >= max_seq) {
        if (ctl && j == 0) ctl[CTL_STATUS] = DEV_POS_OVERFLOW;
        return;
    }
    int width = (Hq + 2 * Hkv) * hd;
    const float* src = qkv + (size_t)m * width + (size_t)h * hd;
    float a = src[j], b = src[j + half];
    if (h < Hq + Hkv) {
        float f = inv_freq ? inv_freq[j] : (float)pow((double)theta, -2.0 * (double)j / (double)hd);
        float s, c;
        sincosf((float)pos * f, &s, &c);
        float ra = a * c - b * s;
        float rb = a * s + b * c;
        a = ra;
        b = rb;
    }
    uint16_t* dst;
    if (h < Hq) {
        dst = q_out + (size_t)m * Hq * hd + (size_t)h * hd;
    } else if (h < Hq + Hkv) {
        dst = kpages + kv_row_offset(page_table, pos, page_shift, Hkv, h - Hq, hd);
    } else {
        dst = vpages + kv_row_offset(page_table, pos, page_shift, Hkv, h - Hq - Hkv, hd);
    }
    dst[j] = f2bf(a);
    dst[j + half] = f2bf(b);
}

// ------------------------------------------------------------------ attention
// grid (chunks, Hkv), block 256.  CTA = keys [64*ch, 64*ch + 64) of KV head kh, all
// G = Hq/Hkv query heads of the group, all M rows.  Row m at position pos0+m sees keys
// <= pos0+m.  Every CTA writes, per (row, head, chunk), the un-normalised partial
// (o[HD], max, sum); the CTA that finishes last for its KV head (a counter, no waiting)
// merges the chunks of that head's queries IN CHUNK ORDER and writes the bf16 output.
// Chunks are cut by absolute position, so a row's result depends on its position only.
//
// q.k and p.v run on the tensor cores (mma.sync.m16n8k16, fp32 accumulate) at EVERY pass size,
// one row or sixteen: queries are the 16-row operand (tiles of 16, zero-padded), so the
// instruction sequence behind a row does not depend on M.  q.k: warp w owns keys 8w..8w+7;
// a thread's 16-byte pieces of its query rows and of its key row are its fragments (the
// contraction index is permuted alike on both sides).  p.v: p is rounded to bf16, warp w owns
// 16 (HD 128) or 8 (HD 64) output dims, V fragments come transposed out of ldmatrix.
// Row pitches keep every access pattern free of bank conflicts: K and Q rows 64 mod 128
// bytes, V rows 16 mod 128 bytes.
//
// shared memory: Ks [64][HD*2+64 B] | Vs [64][HD*2+16 B] | Qb bf16 [Qpad][HD*2+64 B]
//                | S f32 [Qpad][72] | Pb bf16 [Qpad][72]          (Qpad = Q rounded up to 16)
constexpr int kAttnThreads = 256;
constexpr int kAttnMaxChunks = 256;  // chunks the merge can hold weights for: max_seq <= 16384
constexpr int kMergeBatch = 8;       // queries merged together (one warp each)
constexpr int kAttnSP = 72;          // floats per row of S, bf16 per row of Pb
template <int HD>
__host__ __device__ constexpr size_t attn_smem_bytes(int Q)
{
    const size_t qpad = ((size_t)Q + 15) / 16 * 16;
    size_t stage = (size_t)kAttnChunk * (HD * 2 + 64) + (size_t)kAttnChunk * (HD * 2 + 16) + qpad * (HD * 2 + 64) +
                   qpad * kAttnSP * 4 + qpad * kAttnSP * 2;
    // merge (reuses the same memory): weights and sums [8][256] each, slice sums [4][8 slices][HD]
    size_t merge = sizeof(float) * (2 * (size_t)kMergeBatch * kAttnMaxChunks + 4 * 8 * (size_t)HD + kMergeBatch);
    return stage > merge ? stage : merge;
}
// floats per (row, head, chunk) partial: o[HD], max, sum, 2 of padding (16-byte rows)
__host__ __device__ constexpr int attn_part_pitch(int hd) { return hd + 4; }

// scores of QB queries against the thread's key: its quarter of the dims
template <int HD, int QB>
__device__ __forceinline__ void attn_qk(const unsigned char* krow, const float* Qs, int q0, int qd, float* S,
                                        int key, int lane_is_writer)
{
    constexpr int NB = HD / 32;  // 16-byte blocks of the key row per lane
    float acc[QB];
#pragma unroll
    for (int qq = 0; qq < QB; ++qq) acc[qq] = 0.f;
#pragma unroll
    for (int i = 0; i < NB; ++i) {
        const int blk = 4 * i + qd;
        const uint4 kk = *reinterpret_cast<const uint4*>(krow + blk * 16);
        const float kf[8] = {bf16lo(kk.x), bf16hi(kk.x), bf16lo(kk.y), bf16hi(kk.y),
                             bf16lo(kk.z), bf16hi(kk.z), bf16lo(kk.w), bf16hi(kk.w)};
#pragma unroll
        for (int qq = 0; qq < QB; ++qq) {
            const float4* qv = reinterpret_cast<const float4*>(Qs + (size_t)(q0 + qq) * HD + blk * 8);
            const float4 a = qv[0], c = qv[1];
            float s = acc[qq];
            s = fmaf(kf[0], a.x, s);
            s = fmaf(kf[1], a.y, s);
            s = fmaf(kf[2], a.z, s);
            s = fmaf(kf[3], a.w, s);
            s = fmaf(kf[4], c.x, s);
            s = fmaf(kf[5], c.y, s);
            s = fmaf(kf[6], c.z, s);
            s = fmaf(kf[7], c.w, s);
            acc[qq] = s;
        }
    }
#pragma unroll
    for (int qq = 0; qq < QB; ++qq) {
        float s = acc[qq];
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (lane_is_writer) S[(size_t)(q0 + qq) * kAttnChunk + key] = s;
    }
}

// weighted values of QB queries for the thread's pair of dims: its slice of the keys
template <int HD, int QB, int NKS>
__device__ __forceinline__ void attn_pv(const unsigned char* Vs, const float* P, int q0, int dp, int ks,
                                        float (&o)[QB][2])
{
    constexpr int VROW = HD * 2 + 32;
#pragma unroll
    for (int qq = 0; qq < QB; ++qq) o[qq][0] = o[qq][1] = 0.f;
#pragma unroll 4
    for (int j = ks; j < kAttnChunk; j += NKS) {
        const uint32_t u = *reinterpret_cast<const uint32_t*>(Vs + j * VROW + dp * 4);
        const float v0 = bf16lo(u), v1 = bf16hi(u);
#pragma unroll
        for (int qq = 0; qq < QB; ++qq) {
            const float p = P[(size_t)(q0 + qq) * kAttnChunk + j];
            o[qq][0] = fmaf(p, v0, o[qq][0]);
            o[qq][1] = fmaf(p, v1, o[qq][1]);
        }
    }
#pragma unroll
    for (int qq = 0; qq < QB; ++qq)
#pragma unroll
        for (int sh = 1; sh < NKS; sh <<= 1) {
            o[qq][0] += __shfl_xor_sync(0xffffffffu, o[qq][0], sh);
            o[qq][1] += __shfl_xor_sync(0xffffffffu, o[qq][1], sh);
        }
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads)
attn_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ kpages,
            const uint16_t* __restrict__ vpages, const int32_t* __restrict__ page_table,
            int32_t* ctl, int pos_off, int M, int Hq, int Hkv, int page_shift,
            int max_seq, int chunk_cap, float* part, int32_t* counters, uint16_t* __restrict__ out, int gate)
{
    constexpr int C = kAttnChunk, T = kAttnThreads;
    constexpr int KROW = HD * 2 + 64, VROW = HD * 2 + 16;
    constexpr int SP = kAttnSP, PBROW = kAttnSP * 2;
    constexpr int SEGS = HD * 2 / 16;  // 16-byte segments per row
    constexpr int PP = attn_part_pitch(HD);
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned char* Ks = smem;
    unsigned char* Vs = Ks + C * KROW;
    const int ch = blockIdx.x, kh = blockIdx.y, tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    const int key0 = ch * C;
    const uint32_t ks0 = (uint32_t)__cvta_generic_to_shared(Ks), vs0 = (uint32_t)__cvta_generic_to_shared(Vs);
    const bool one_page = page_shift >= 6;

    // Cache rows below the loop's cache length do not change while the loop runs, so their
    // copies start before the producer of q (and of this pass's own k, v rows) has finished.
    // The length is read past L1 and may be an older, smaller one: then fewer rows go early.
    pdl_launch_dependents();
    int c_early = 0;
    if (ctl && !(gate > 0 && gate > __ldcg(ctl + CTL_D_EFF))) c_early = min(__ldcg(ctl + CTL_CACHE_LEN), max_seq);
    size_t base = 0;
    auto stage_rows = [&](int p_lo, int p_hi, int p_fill) {
        // rows p of the chunk with p_lo <= p <= p_hi are copied; rows p_hi < p <= p_fill are zeroed
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
    if (key0 < c_early) {
        if (one_page) base = kv_row_offset(page_table, key0, page_shift, Hkv, kh, HD);
        stage_rows(0, c_early - 1, c_early - 1);
    }
    pdl_wait();
    auto leave = [&]() {  // nothing in flight may outlive the CTA's shared memory
        cp_async_commit();
        cp_async_wait<0>();
    };
    if (pass_idle(ctl, gate)) return leave();
    const int pos0 = (ctl ? ctl[CTL_CACHE_LEN] : 0) + pos_off;
    const int last_pos = pos0 + M - 1;
    if (key0 > last_pos) return leave();
    const int n_active = last_pos / C + 1;  // CTAs of this KV head that take part
    if (last_pos >= max_seq || pos0 < 0 || n_active > chunk_cap || n_active > (int)gridDim.x) {
        if (ctl && tid == 0) ctl[CTL_STATUS] = DEV_POS_OVERFLOW;
        return leave();
    }
    if (c_early > pos0) c_early = pos0;  // (cannot happen: the length only grows; rows >= pos0 are this pass's)
    const int G = Hq / Hkv, Q = G * M;  // query qi = m * G + g
    const int Qpad = (Q + 15) & ~15;

    unsigned char* Qb = Vs + C * VROW;
    float* S = reinterpret_cast<float*>(Qb + (size_t)Qpad * KROW);
    unsigned char* Pb = reinterpret_cast<unsigned char*>(S + (size_t)Qpad * SP);

    // the group's queries (bf16, 16-byte pieces): issue the global loads first, so that they
    // travel together with the page-table lookup and the K/V copies
    constexpr int QPT = 2;
    const int nq = Qpad * SEGS;
    uint4 qreg[QPT];
#pragma unroll
    for (int i = 0; i < QPT; ++i) {
        const int idx = tid + i * T;
        qreg[i] = make_uint4(0, 0, 0, 0);
        if (idx < nq) {
            const int qi = idx / SEGS, sg = idx % SEGS;
            if (qi < Q) {
                const int m = qi / G, g = qi % G;
                qreg[i] = *reinterpret_cast<const uint4*>(q + ((size_t)m * Hq + (size_t)kh * G + g) * HD + sg * 8);
            }
        }
    }
    // stage the remaining K and V rows of the chunk (zeros beyond the last visible key):
    // asynchronous copies, all in flight at once; a chunk never straddles a page of 64 tokens
    // or more
    if (one_page) base = kv_row_offset(page_table, key0, page_shift, Hkv, kh, HD);
    stage_rows(c_early, last_pos, key0 + C - 1);
    cp_async_commit();
#pragma unroll
    for (int i = 0; i < QPT; ++i) {
        const int idx = tid + i * T;
        if (idx < nq) *reinterpret_cast<uint4*>(Qb + (idx / SEGS) * KROW + (idx % SEGS) * 16) = qreg[i];
    }
    for (int idx = tid + QPT * T; idx < nq; idx += T) {  // more than two tiles of queries
        const int qi = idx / SEGS, sg = idx % SEGS;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (qi < Q) {
            const int m = qi / G, g = qi % G;
            v = *reinterpret_cast<const uint4*>(q + ((size_t)m * Hq + (size_t)kh * G + g) * HD + sg * 8);
        }
        *reinterpret_cast<uint4*>(Qb + qi * KROW + sg * 16) = v;
    }
    cp_async_wait<0>();
    __syncthreads();

    // phase 1: s = q.k -- warp w: keys 8w..8w+7 against every tile of 16 queries
    for (int qt = 0; qt < Qpad; qt += 16) {
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
        float* s = S + (size_t)(qt + g8) * SP + 8 * warp + 2 * t4;
        *reinterpret_cast<float2*>(s) = make_float2(c[0], c[1]);
        *reinterpret_cast<float2*>(s + 8 * SP) = make_float2(c[2], c[3]);
    }
    __syncthreads();

    // phase 2: one warp per query: scale, mask, max, exp, sum over the 64 keys of the chunk;
    // p goes to Pb as bf16 (zeros for the padding rows of the last tile)
    {
        const float scale = rsqrtf((float)HD);
        for (int qi = warp; qi < Qpad; qi += T / 32) {
            uint16_t* pb = reinterpret_cast<uint16_t*>(Pb + (size_t)qi * PBROW);
            if (qi >= Q) {
                pb[lane] = 0;
                pb[lane + 32] = 0;
                continue;
            }
            const int m = qi / G, g = qi % G;
            const int pos = pos0 + m;
            float s0 = S[(size_t)qi * SP + lane] * scale;
            float s1 = S[(size_t)qi * SP + lane + 32] * scale;
            if (key0 + lane > pos) s0 = -INFINITY;
            if (key0 + lane + 32 > pos) s1 = -INFINITY;
            float mx = fmaxf(s0, s1);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float p0 = (s0 == -INFINITY) ? 0.f : expf(s0 - mx);
            const float p1 = (s1 == -INFINITY) ? 0.f : expf(s1 - mx);
            float l = p0 + p1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            pb[lane] = f2bf(p0);
            pb[lane + 32] = f2bf(p1);
            if (lane == 0) {
                float* dst = part + (((size_t)m * Hq + (size_t)kh * G + g) * chunk_cap + ch) * PP;
                dst[HD] = mx;
                dst[HD + 1] = l;
            }
        }
    }
    __syncthreads();

    // phase 3: o = p.v -- warp w: output dims NTW*8*w .. for every tile of 16 queries
    {
        constexpr int NTW = HD / 64;  // n8 tiles per warp: 2 (HD 128) or 1 (HD 64)
        const int d0 = NTW * 8 * warp;
        const uint32_t vs0 = (uint32_t)__cvta_generic_to_shared(Vs);
        // ldmatrix: lane L addresses row L%8 of matrix L/8; matrices 0, 1: keys 0-7, 8-15 of
        // the 16-key block at dims d0..d0+7; matrices 2, 3: the same keys at dims d0+8..
        const int mi = lane >> 3, mr = lane & 7;
        const uint32_t vlane = vs0 + (uint32_t)(((mi & 1) * 8 + mr) * VROW + (d0 + ((NTW == 2) ? (mi >> 1) * 8 : 0)) * 2);
        for (int qt = 0; qt < Qpad; qt += 16) {
            float c[NTW][4];
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) c[nt][i] = 0.f;
            const unsigned char* pa = Pb + (size_t)(qt + g8) * PBROW + 4 * t4;
#pragma unroll
            for (int kk = 0; kk < C / 16; ++kk) {
                const uint32_t a0 = *reinterpret_cast<const uint32_t*>(pa + 32 * kk);
                const uint32_t a1 = *reinterpret_cast<const uint32_t*>(pa + 8 * PBROW + 32 * kk);
                const uint32_t a2 = *reinterpret_cast<const uint32_t*>(pa + 32 * kk + 16);
                const uint32_t a3 = *reinterpret_cast<const uint32_t*>(pa + 8 * PBROW + 32 * kk + 16);
                uint32_t r0, r1, r2, r3;
                ldmatrix_x4_trans(vlane + (uint32_t)(16 * kk * VROW), r0, r1, r2, r3);
                mma_bf16_16816(c[0], a0, a1, a2, a3, r0, r1);
                if (NTW == 2) mma_bf16_16816(c[NTW - 1], a0, a1, a2, a3, r2, r3);
            }
#pragma unroll
            for (int hrow = 0; hrow < 2; ++hrow) {
                const int qi = qt + g8 + 8 * hrow;
                if (qi < Q) {
                    const int m = qi / G, g = qi % G;
                    float* dst = part + (((size_t)m * Hq + (size_t)kh * G + g) * chunk_cap + ch) * PP + d0 + 2 * t4;
#pragma unroll
                    for (int nt = 0; nt < NTW; ++nt)
                        *reinterpret_cast<float2*>(dst + 8 * nt) = make_float2(c[nt][2 * hrow], c[nt][2 * hrow + 1]);
                }
            }
        }
    }

    // who is last for this KV head?  (publish the partials, then count; nobody waits)
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(&counters[kh], 1);
        is_last = (prev == n_active - 1);
        if (is_last) counters[kh] = 0;  // ready for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // Merge in a fixed order, in two round trips to L2 per batch of 8 queries:
    //  A  one warp per query: all chunk (max, sum) pairs at once -> global max, weights
    //     w_c = exp(max_c - max) and the denominator (summed in chunk order by one lane);
    //  B  four queries at a time: warp s sums the weighted o of chunks c = s, s+8, ... of each
    //     (lanes over the dims), then one warp per query adds the 8 slice sums in slice
    //     order, divides and stores.
    // The order depends on the row's position only, never on M.
    {
        constexpr int DPL = HD / 32;  // dims per lane: 4 or 2
        const int warp = tid >> 5, lane = tid & 31;
        float* Wt = reinterpret_cast<float*>(smem);                 // [8][kAttnMaxChunks] weights
        float* Ls = Wt + kMergeBatch * kAttnMaxChunks;              // [8][kAttnMaxChunks] chunk sums
        float* Ob = Ls + kMergeBatch * kAttnMaxChunks;              // [4 queries][8 slices][HD]
        float* Lq = Ob + 4 * 8 * HD;                                // [8] denominators
        for (int qb = 0; qb < Q; qb += kMergeBatch) {
            __syncthreads();  // previous batch (and the phases before) are done with this memory
            {
                const int qi = qb + warp;
                if (qi < Q) {
                    const int m = qi / G, h = kh * G + qi % G;
                    const int nch = (pos0 + m) / C + 1;
                    const float* base = part + ((size_t)m * Hq + h) * chunk_cap * PP;
                    float* wt = Wt + warp * kAttnMaxChunks;
                    float* ls = Ls + warp * kAttnMaxChunks;
                    float mx = -INFINITY;
                    for (int c = lane; c < nch; c += 32) {
                        const float2 ml = __ldcg(reinterpret_cast<const float2*>(base + (size_t)c * PP + HD));
                        wt[c] = ml.x;
                        ls[c] = ml.y;
                        mx = fmaxf(mx, ml.x);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    for (int c = lane; c < nch; c += 32) wt[c] = expf(wt[c] - mx);
                    __syncwarp();
                    if (lane == 0) {
                        float l = 0.f;
                        for (int c = 0; c < nch; ++c) l = fmaf(ls[c], wt[c], l);
                        Lq[warp] = l;
                    }
                }
            }
            __syncthreads();
            for (int w0 = 0; w0 < kMergeBatch && qb + w0 < Q; w0 += 4) {  // four queries at a time
                float o[4][DPL];
#pragma unroll
                for (int ww = 0; ww < 4; ++ww) {
#pragma unroll
                    for (int i = 0; i < DPL; ++i) o[ww][i] = 0.f;
                    const int qi = qb + w0 + ww;
                    if (qi < Q) {
                        const int m = qi / G, h = kh * G + qi % G;
                        const int nch = (pos0 + m) / C + 1;
                        const float* base = part + ((size_t)m * Hq + h) * chunk_cap * PP + lane * DPL;
                        const float* wt = Wt + (w0 + ww) * kAttnMaxChunks;
#pragma unroll 4
                        for (int c = warp; c < nch; c += 8) {
                            const float wc = wt[c];
                            if (DPL == 4) {
                                const float4 v = __ldcg(reinterpret_cast<const float4*>(base + (size_t)c * PP));
                                o[ww][0] = fmaf(v.x, wc, o[ww][0]);
                                o[ww][1] = fmaf(v.y, wc, o[ww][1]);
                                o[ww][DPL - 2] = fmaf(v.z, wc, o[ww][DPL - 2]);
                                o[ww][DPL - 1] = fmaf(v.w, wc, o[ww][DPL - 1]);
                            } else {
                                const float2 v = __ldcg(reinterpret_cast<const float2*>(base + (size_t)c * PP));
                                o[ww][0] = fmaf(v.x, wc, o[ww][0]);
                                o[ww][1] = fmaf(v.y, wc, o[ww][1]);
                            }
                        }
                    }
                }
#pragma unroll
                for (int ww = 0; ww < 4; ++ww)
#pragma unroll
                    for (int i = 0; i < DPL; ++i) Ob[(ww * 8 + warp) * HD + lane * DPL + i] = o[ww][i];
                __syncthreads();
                if (warp < 4 && qb + w0 + warp < Q) {  // warp ww finishes query w0 + ww
                    const int qi = qb + w0 + warp;
                    const int m = qi / G, h = kh * G + qi % G;
                    const float l = Lq[w0 + warp];
                    float r[DPL];
#pragma unroll
                    for (int i = 0; i < DPL; ++i) {
                        float a = 0.f;
#pragma unroll
                        for (int sl = 0; sl < 8; ++sl) a += Ob[(warp * 8 + sl) * HD + lane * DPL + i];
                        r[i] = a / l;
                    }
                    uint16_t* dst = out + ((size_t)m * Hq + h) * HD + lane * DPL;
                    if (DPL == 4) {
                        uint2 pk;
                        pk.x = pack_bf16(r[0], r[1]);
                        pk.y = pack_bf16(r[DPL - 2], r[DPL - 1]);
                        *reinterpret_cast<uint2*>(dst) = pk;
                    } else {
                        *reinterpret_cast<uint32_t*>(dst) = pack_bf16(r[0], r[1]);
                    }
                }
                __syncthreads();
            }
        }
    }
}

// ------------------------------------------------------------------ argmax finish
// grid M, block 256: reduce the per-CTA (value, index) candidates of the LM-head kernel.
// (value desc, index asc) is a total order, so the result does not depend on the
// reduction tree; the lowest index wins a tie.
// Adaptive drafting (second != nullptr; the launch is the head of draft pass `gate`, M = 1):
// the per-CTA second-largest logits are reduced too, and when the margin between the two
// largest exit logits is below min_margin this draft is not kept and drafting stops:
// CTL_D_EFF = gate, which idles every later draft pass of the step.  Where the step is a CUDA
// graph whose later draft passes are conditional nodes, next_pass is the handle of the next
// pass's node (0: none): it is switched on only when this draft is kept.
__global__ void __launch_bounds__(256)
argmax_finish_kernel(const ValIdx* __restrict__ cand, int n_cand, int cand_stride,
                     int32_t* __restrict__ tok_out, int32_t* ctl, const float* __restrict__ second,
                     float min_margin, int gate, unsigned long long next_pass)
{
    __shared__ float sv[256];
    __shared__ float s2[256];
    __shared__ int si[256];
    pdl_launch_dependents();
    pdl_wait();
    if (pass_idle(ctl, gate)) return;
    int m = blockIdx.x;
    const ValIdx* c = cand + (size_t)m * cand_stride;
    float bv = -INFINITY, bs = -INFINITY;
    int bi = 0x7fffffff;
    for (int k = threadIdx.x; k < n_cand; k += 256) {
        ValIdx e = c[k];
        top2_merge(e.v, e.i, second ? second[(size_t)m * cand_stride + k] : -INFINITY, bv, bi, bs);
    }
    sv[threadIdx.x] = bv;
    s2[threadIdx.x] = bs;
    si[threadIdx.x] = bi;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
            top2_merge(sv[threadIdx.x + s], si[threadIdx.x + s], s2[threadIdx.x + s], bv, bi, bs);
            sv[threadIdx.x] = bv;
            s2[threadIdx.x] = bs;
            si[threadIdx.x] = bi;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        tok_out[m] = bi;
        if (second && ctl && m == 0) {
            if (bv - bs < min_margin) {
                if (gate < ctl[CTL_D_EFF]) ctl[CTL_D_EFF] = gate;
            } else if (next_pass) {
                cudaGraphSetConditional((cudaGraphConditionalHandle)next_pass, 1);
            }
        }
    }
}

// ------------------------------------------------------------------ accept / rollback
// match + crop of the paper's loop (Appendix A.4), one thread.  With d == 0 it is the
// bookkeeping of plain greedy decoding (emit verified[0]).  Adaptive drafting (adaptive != 0):
// only the drafts the step kept (CTL_D_EFF of them) can be accepted; their number goes to
// drafted[step] and the stop mark is cleared for the next step.
__global__ void accept_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ verified,
                              int d, int32_t* ctl, int32_t* __restrict__ out_ids,
                              int32_t* __restrict__ accepted, int adaptive, int32_t* __restrict__ drafted)
{
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    if (ctl[CTL_DONE]) return;
    if (adaptive) {
        d = min(d, ctl[CTL_D_EFF]);
        ctl[CTL_D_EFF] = kNoStop;
    }
    int n = 0;
    while (n < d && draft[n] == verified[n]) ++n;
    int n_out = ctl[CTL_N_OUT];
    const int max_new = ctl[CTL_MAX_NEW], eos = ctl[CTL_EOS];
    bool stop = false;
    for (int i = 0; i <= n && n_out < max_new && !stop; ++i) {
        int t = (i < n) ? draft[i] : verified[n];
        out_ids[n_out++] = t;
        if (eos >= 0 && t == eos) stop = true;
    }
    int steps = ctl[CTL_N_STEPS];
    accepted[steps] = n;
    if (drafted) drafted[steps] = d;
    ctl[CTL_N_STEPS] = steps + 1;
    ctl[CTL_N_OUT] = n_out;
    ctl[CTL_CUR_TOK] = verified[n];
    ctl[CTL_CACHE_LEN] += n + 1;
    if (stop || n_out >= max_new) ctl[CTL_DONE] = 1;
}

}  // namespace ls

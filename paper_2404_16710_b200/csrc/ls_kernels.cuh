// Non-GEMV kernels of the decode loop: embedding, RMSNorm, rotary embedding + KV append,
// argmax finish, accept/rollback (attention: ls_attention.cuh).
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
// grid M, block 256.  tok[m * tok_stride] is read from device memory (stride CTL_WORDS: the
// current tokens in the sequences' control blocks).  With gain != nullptr the kernel
// also leaves what the first layer's fused RMSNorm needs: hout = bf16(x * gain) and the
// row's exact sum of squares (ls_common.cuh) in slot 0 of ss_out[m][kSsSlots] (the other slots zero).
__global__ void __launch_bounds__(256)
embed_kernel(const uint16_t* __restrict__ emb, const int32_t* __restrict__ tok, int D, int V,
             float* __restrict__ x, int32_t* ctl, const uint16_t* __restrict__ gain,
             uint16_t* __restrict__ hout, long long* __restrict__ ss_out, int gate, int tok_stride)
{
    __shared__ long long red[8];
    pdl_launch_dependents();
    pdl_wait();
    if (pass_idle(ctl, gate)) return;
    int m = blockIdx.x;
    int id = tok[(size_t)m * tok_stride];
    if (id < 0 || id >= V) {
        if (ctl && threadIdx.x == 0) ctl[CTL_STATUS] = DEV_BAD_TOKEN;
        id = 0;
    }
    const uint4* src = reinterpret_cast<const uint4*>(emb + (size_t)id * D);
    float4* dst = reinterpret_cast<float4*>(x + (size_t)m * D);
    long long ss = 0;
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
            for (int e = 0; e < 8; ++e) ss += sq_fixed(f[e]);
        }
    }
    if (gain) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x < kSsSlots) {
            long long tot = 0;
            if (threadIdx.x == 0) {
#pragma unroll
                for (int w = 0; w < 8; ++w) tot += red[w];
            }
            ss_out[(size_t)m * kSsSlots + threadIdx.x] = tot;
        }
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

// ------------------------------------------------------------------ attention: shared constants
// (the decode / verify kernel is in ls_attention.cuh; the two helpers below serve the FMA walk
// of the prompt pass)
constexpr int kAttnThreads = 256;
constexpr int kAttnMaxChunks = 256;  // chunks of 64 keys a cache may hold: max_seq <= 16384
constexpr int kAttnSP = 72;          // floats per row of S, bf16 per row of Pb

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

// The same bookkeeping for B sequences that share every pass (thread b: sequence b).  draft and
// verified are laid out [position][sequence]; sequence b emits into out_ids + b * out_stride
// and records into accepted + b * out_stride; a sequence that has finished is left alone (its
// rows keep running through the passes, nobody reads them).  CTL_DONE of block 0 is set once
// every sequence has finished.
__global__ void accept_batch_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ verified,
                                    int d, int B, int32_t* ctl, int32_t* __restrict__ out_ids,
                                    int32_t* __restrict__ accepted, int out_stride)
{
    pdl_launch_dependents();
    pdl_wait();
    if (blockIdx.x != 0 || ctl[CTL_DONE]) return;
    const int b = threadIdx.x;
    bool finished = true;
    if (b < B) {
        int32_t* c = ctl + b * CTL_WORDS;
        finished = c[CTL_SEQ_DONE] != 0;
        if (!finished) {
            int n = 0;
            while (n < d && draft[n * B + b] == verified[n * B + b]) ++n;
            int n_out = c[CTL_N_OUT];
            const int max_new = c[CTL_MAX_NEW], eos = c[CTL_EOS];
            bool stop = false;
            for (int i = 0; i <= n && n_out < max_new && !stop; ++i) {
                const int t = (i < n) ? draft[i * B + b] : verified[n * B + b];
                out_ids[(size_t)b * out_stride + n_out++] = t;
                if (eos >= 0 && t == eos) stop = true;
            }
            const int steps = c[CTL_N_STEPS];
            accepted[(size_t)b * out_stride + steps] = n;
            c[CTL_N_STEPS] = steps + 1;
            c[CTL_N_OUT] = n_out;
            c[CTL_CUR_TOK] = verified[n * B + b];
            c[CTL_CACHE_LEN] += n + 1;
            if (stop || n_out >= max_new) {
                c[CTL_SEQ_DONE] = 1;
                finished = true;
            }
        }
    }
    if (__syncthreads_and(finished) && threadIdx.x == 0) ctl[CTL_DONE] = 1;
}

}  // namespace ls

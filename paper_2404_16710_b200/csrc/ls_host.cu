// Host side of the library: model handle, workspace carve-up, the draft / verify /
// accept schedule of LayerSkip's self-speculative decoding (Sec. 4.3, Appendix A.4)
// as CUDA graphs, and the C ABI declared in ls.h.
//
// Schedule of one speculative step (E early layers, d drafts), all on one stream, all
// positions read by the kernels from the control words in device memory:
//   for j = 0..d:   embed(input_j) -> layers 0..E-1 on residual row j at position c+j
//                   (j < d: final norm + LM head + argmax -> draft[j] = input_{j+1})
//   verify:         layers E..L-1 on residual rows 0..d (they ARE the exit-layer
//                   activations: nothing is copied), final norm + LM head + argmax
//   accept:         match, emit, crop (one tiny kernel); sets the done flag
// The host launches a batch of step graphs sized to the tokens still missing and only
// then looks at the control words, so there is no host sync per token; steps launched
// past the end see the done flag and return at once.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <tuple>
#include <mutex>
#include <new>
#include <vector>

#include "ls.h"
#include "ls_attention.cuh"
#include "ls_linear.cuh"
#include "ls_prefill.cuh"
#include "ls_prefill_attn.cuh"

using namespace ls;

namespace {

thread_local int g_last_cuda = 0;
bool g_op_chain = false;  // ls_op_* launches carry the programmatic-dependent-launch attribute (ls_op_chain)

#define LS_CK(expr)                         \
    do {                                    \
        cudaError_t e_ = (expr);            \
        if (e_ != cudaSuccess) {            \
            g_last_cuda = (int)e_;          \
            return LS_ERR_CUDA;             \
        }                                   \
    } while (0)

#define LS_TRY(expr)            \
    do {                        \
        int rc_ = (expr);       \
        if (rc_ != LS_OK) return rc_; \
    } while (0)

constexpr int kPrefillBlock = 1024;  // rows the prompt pass handles at a time

struct LayerW {
    const uint16_t *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *wg, *wu, *wd;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return p && ((uintptr_t)p & 15u) == 0; }

int log2_exact(int v)
{
    int s = 0;
    while ((1 << s) < v) ++s;
    return ((1 << s) == v) ? s : -1;
}

bool config_ok(const ls_config* c)
{
    if (!c) return false;
    if (c->n_layers < 1 || c->d_model < 8 || c->d_model % 8 || c->d_ffn < 8 || c->d_ffn % 8) return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->n_heads < 1 || c->n_kv_heads < 1 || c->n_heads % c->n_kv_heads) return false;
    if (c->n_heads / c->n_kv_heads > 8) return false;
    if (c->vocab < 1 || c->max_seq < 2 || c->max_seq > kAttnChunk * kAttnMaxChunks) return false;
    if (c->page_size < 16 || c->page_size > 1024 || log2_exact(c->page_size) < 0) return false;
    if (c->max_draft < 0 || c->max_draft + 1 > LS_MAX_ROWS) return false;
    if (c->linear_path < 0 || c->linear_path > 2) return false;
    if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 0.f)) return false;
    return true;
}

}  // namespace

struct ls_model {
    ls_config c;
    int path;
    cudaStream_t st;
    std::vector<LayerW> lw;
    const uint16_t *emb, *fnorm, *lm;
    // workspace
    uint16_t *kpages, *vpages;
    size_t layer_kv_elems;
    int32_t *page_table, *ctl, *draft, *verified, *out_ids, *accepted, *ids;
    float *inv_freq, *x, *logits;
    float2* rope_tab;  // (cos, sin) of every position and rotary pair, for the prompt pass's q|k|v epilogue
    uint16_t *h, *q, *o, *a;
    uint16_t* hE;  // exit-layer activations, already multiplied by the gain of layer E's norm (Sec. 4.3.3)
    float *px, *py;          // prompt pass: residual rows and projection outputs of one block
    uint16_t *ph, *pq, *po, *pa;
    // exact sums of squares of the residual rows (fused RMSNorm), [16][kSsSlots] each: after the
    // attention block (o-proj adds, gate-up reads) and after the FFN or the embedding (down-proj
    // adds, q|k|v and the LM head read)
    long long *ss_attn, *ss_ffn;
    ValIdx* cand;
    float* second;      // per-CTA second-largest logit beside each argmax candidate (adaptive drafting)
    int32_t* drafted;   // drafts kept per step (adaptive drafting)
    int gate;           // draft pass the launches being enqueued belong to (0: none)
    unsigned long long next_pass;  // conditional-node handle the next draft head switches on (0: none)
    int page_shift, n_pages, cand_stride;
    AttnPlan attn;  // cluster size and chunks per CTA of the attention kernel: constants of the model
    // The sequences the passes being enqueued carry (ls_common.cuh): their number, the page-table
    // entries and the cache capacity of each, and the table entry of the first.  One sequence
    // owns the whole table; B sequences get n_pages / B pages each.
    int nseq, pt_stride, seq_cap;
    const int32_t* pt;
    std::vector<int> b_n_prompt, b_last_tok;               // several sequences: prompt length and last prompt token of each
    std::vector<std::vector<int32_t>> b_out, b_acc;        // ... and what the last ls_decode_batch produced
    // loop state
    int n_prompt, last_tok, prefilled_layers;
    bool use_graphs, own_stream, pdl, big_prefill, cond_graphs;
    int64_t launches;  // kernels enqueued (counted while building a step)
    struct G {
        cudaGraphExec_t exec;
        int64_t nodes;
    };
    std::map<std::pair<uint64_t, uint32_t>, G> graphs;
    cudaEvent_t ev0, ev1;
    ls_stats stats;
    std::vector<int32_t> h_out, h_acc, h_drafted;
    int h_n_out, h_n_steps;
};

namespace {

// carve the workspace; with base == nullptr only sizes are computed
size_t carve(const ls_config& c, unsigned char* base, ls_model* m)
{
    size_t off = 0;
    auto take = [&](size_t bytes) {
        unsigned char* p = base ? base + off : nullptr;
        off = align_up(off + bytes, 256);
        return p;
    };
    const int n_pages = (c.max_seq + c.page_size - 1) / c.page_size;
    const int cand_stride = (c.vocab + 15) / 16;
    const size_t layer_kv = (size_t)n_pages * c.n_kv_heads * c.page_size * c.head_dim;
    const size_t qw = (size_t)c.n_heads * c.head_dim, kvw = (size_t)c.n_kv_heads * c.head_dim;
    unsigned char* kp = take(layer_kv * c.n_layers * 2);
    unsigned char* vp = take(layer_kv * c.n_layers * 2);
    unsigned char* pt = take(sizeof(int32_t) * n_pages);
    unsigned char* fr = take(sizeof(float) * (c.head_dim / 2));
    unsigned char* rt = take(sizeof(float2) * (size_t)c.max_seq * (c.head_dim / 2));
    unsigned char* ctl = take(sizeof(int32_t) * CTL_WORDS * kMaxRows);  // one block per sequence of a pass
    unsigned char* dr = take(sizeof(int32_t) * kMaxRows);
    unsigned char* ve = take(sizeof(int32_t) * kMaxRows);
    // outputs: sequence b of a pass of several writes from b * (its share of the pages' positions) on
    unsigned char* oi = take(sizeof(int32_t) * (size_t)n_pages * c.page_size);
    unsigned char* ac = take(sizeof(int32_t) * (size_t)n_pages * c.page_size);
    unsigned char* ids = take(sizeof(int32_t) * c.max_seq);
    unsigned char* x = take(sizeof(float) * kMaxRows * c.d_model);
    unsigned char* logits = take(sizeof(float) * kMaxRows * c.vocab);
    unsigned char* h = take(2 * (size_t)kMaxRows * c.d_model);
    unsigned char* q = take(2 * (size_t)kMaxRows * qw);
    unsigned char* o = take(2 * (size_t)kMaxRows * qw);
    unsigned char* a = take(2 * (size_t)kMaxRows * c.d_ffn);
    unsigned char* cand = take(sizeof(ValIdx) * kMaxRows * cand_stride);
    unsigned char* second = take(sizeof(float) * kMaxRows * cand_stride);
    unsigned char* drafted = take(sizeof(int32_t) * c.max_seq);
    unsigned char* ss = take(sizeof(long long) * kMaxRows * kSsSlots * 2);
    unsigned char* he = take(2 * (size_t)kMaxRows * c.d_model);
    const int pb = c.max_seq < kPrefillBlock ? c.max_seq : kPrefillBlock;  // rows per block of the prompt pass
    const size_t ywide = (qw + 2 * kvw) > 2 * (size_t)c.d_ffn ? (qw + 2 * kvw) : 2 * (size_t)c.d_ffn;
    unsigned char* px = take(sizeof(float) * (size_t)pb * c.d_model);
    unsigned char* ph = take(2 * (size_t)pb * c.d_model);
    unsigned char* py = take(sizeof(float) * (size_t)pb * ywide);
    unsigned char* pq = take(2 * (size_t)pb * qw);
    unsigned char* po = take(2 * (size_t)pb * qw);
    unsigned char* pa = take(2 * (size_t)pb * c.d_ffn);
    if (m) {
        m->px = (float*)px;
        m->ph = (uint16_t*)ph;
        m->py = (float*)py;
        m->pq = (uint16_t*)pq;
        m->po = (uint16_t*)po;
        m->pa = (uint16_t*)pa;
        m->ss_attn = (long long*)ss;
        m->ss_ffn = m->ss_attn + kMaxRows * kSsSlots;
        m->hE = (uint16_t*)he;
        m->kpages = (uint16_t*)kp;
        m->vpages = (uint16_t*)vp;
        m->layer_kv_elems = layer_kv;
        m->page_table = (int32_t*)pt;
        m->inv_freq = (float*)fr;
        m->rope_tab = (float2*)rt;
        m->ctl = (int32_t*)ctl;
        m->draft = (int32_t*)dr;
        m->verified = (int32_t*)ve;
        m->out_ids = (int32_t*)oi;
        m->accepted = (int32_t*)ac;
        m->ids = (int32_t*)ids;
        m->x = (float*)x;
        m->logits = (float*)logits;
        m->h = (uint16_t*)h;
        m->q = (uint16_t*)q;
        m->o = (uint16_t*)o;
        m->a = (uint16_t*)a;
        m->cand = (ValIdx*)cand;
        m->second = (float*)second;
        m->drafted = (int32_t*)drafted;
        m->n_pages = n_pages;
        m->cand_stride = cand_stride;
        m->page_shift = log2_exact(c.page_size);
    }
    return off;
}

// ------------------------------------------------------------------ kernel launch helpers
template <int HD, int QT>
int attn_launch_t(const AttnPlan& plan, const uint16_t* q, const uint16_t* kp, const uint16_t* vp, const int32_t* pt,
                  int32_t* ctl, int pos_off, int M, int Hq, int Hkv, int page_shift, int max_seq, uint16_t* out,
                  const LaunchCtx& lc, int gate, int nseq, int pt_stride)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.csize, Hkv, nseq);
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = attn_smem_bytes<HD>(Hq / Hkv * (M / nseq));
    cfg.stream = lc.st;
    // Load-balancing placement: the hardware may put several CTAs of a cluster on one SM.  With
    // the default (spread) policy, clusters that arrive while the previous kernel is still
    // draining are laid out one CTA per SM, two clusters per GPC, and the other half of the
    // grid only starts when those have finished: attention then runs as two waves.
    cudaLaunchAttribute at[3];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = plan.csize;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
    at[1].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicyLoadBalancing;
    at[2].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[2].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = lc.pdl ? 3 : 2;
    LS_CK(cudaLaunchKernelEx(&cfg, attn_cluster_kernel<HD, QT>, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift,
                             max_seq, out, gate, pt_stride));
    return LS_OK;
}

template <int HD>
int attn_launch_hd(const AttnPlan& plan, const uint16_t* q, const uint16_t* kp, const uint16_t* vp, const int32_t* pt,
                   int32_t* ctl, int pos_off, int M, int Hq, int Hkv, int page_shift, int max_seq, uint16_t* out,
                   const LaunchCtx& lc, int gate, int nseq, int pt_stride)
{
    const int Q = Hq / Hkv * (M / nseq);  // the instantiation that holds a sequence's Q queries in tiles of 16
    if (Q <= 16)
        return attn_launch_t<HD, 1>(plan, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift, max_seq, out, lc, gate, nseq, pt_stride);
    if (Q <= 32)
        return attn_launch_t<HD, 2>(plan, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift, max_seq, out, lc, gate, nseq, pt_stride);
    if (Q <= 64)
        return attn_launch_t<HD, 4>(plan, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift, max_seq, out, lc, gate, nseq, pt_stride);
    return attn_launch_t<HD, 8>(plan, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift, max_seq, out, lc, gate, nseq, pt_stride);
}

int attn_launch(const AttnPlan& plan, const uint16_t* q, const uint16_t* kp, const uint16_t* vp, const int32_t* pt,
                int32_t* ctl, int pos_off, int M, int Hq, int Hkv, int hd, int page_shift, int max_seq, uint16_t* out,
                const LaunchCtx& lc, int gate = 0, int nseq = 1, int pt_stride = 0)
{
    if (hd == 128)
        return attn_launch_hd<128>(plan, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift, max_seq, out, lc, gate, nseq, pt_stride);
    return attn_launch_hd<64>(plan, q, kp, vp, pt, ctl, pos_off, M, Hq, Hkv, page_shift, max_seq, out, lc, gate, nseq, pt_stride);
}

template <int HD, int QT>
cudaError_t attn_prepare_t(int group, int Hkv, int csize, int* clusters)
{
    const int rows = 16 * QT / group;  // rows of the largest pass this instantiation serves
    if (rows < 1) return cudaSuccess;
    const size_t smem = attn_smem_bytes<HD>(group * (rows < kMaxRows ? rows : kMaxRows));
    cudaError_t e = cudaFuncSetAttribute(attn_cluster_kernel<HD, QT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess || !clusters) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(csize, Hkv);
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = csize;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
    at[1].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicyLoadBalancing;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    return cudaOccupancyMaxActiveClusters(clusters, attn_cluster_kernel<HD, QT>, &cfg);
}

template <int HD>
cudaError_t attn_prepare_hd(int group, int Hkv, int csize, int* clusters)
{
    // every instantiation gets its shared-memory allowance; the residency question is asked
    // of the one that serves single-row passes (the bulk of the loop)
    cudaError_t e = attn_prepare_t<HD, 1>(group, Hkv, csize, clusters);
    if (e == cudaSuccess) e = attn_prepare_t<HD, 2>(group, Hkv, csize, nullptr);
    if (e == cudaSuccess) e = attn_prepare_t<HD, 4>(group, Hkv, csize, nullptr);
    if (e == cudaSuccess) e = attn_prepare_t<HD, 8>(group, Hkv, csize, nullptr);
    return e;
}

// Cluster size for a cache of max_seq positions: the largest cluster (up to 8 CTAs, no more
// than the cache has chunks) with which one cluster per KV head is resident at the same time, so
// that no head waits for another to finish; 8 if no size achieves that.  A function of the
// model's shape and the device only -- never of a pass -- because the cluster size decides which
// chunks a CTA folds together, which enters a row's arithmetic.
int attn_plan(int hd, int group, int Hkv, int max_seq, AttnPlan* out)
{
    struct Key {
        int dev, hd, group, Hkv, cap;
        bool operator<(const Key& o) const
        {
            return std::tie(dev, hd, group, Hkv, cap) < std::tie(o.dev, o.hd, o.group, o.Hkv, o.cap);
        }
    };
    static std::map<Key, AttnPlan> plans;
    static std::mutex mu;
    const int cap = (max_seq + kAttnChunk - 1) / kAttnChunk;
    int dev = 0;
    LS_CK(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(mu);
    const Key key = {dev, hd, group, Hkv, cap};
    auto it = plans.find(key);
    if (it == plans.end()) {
        int best = 0;
        const int cmax = cap < kAttnMaxCluster ? cap : kAttnMaxCluster;
        for (int cs = cmax; cs >= 1 && !best; --cs) {
            int clusters = 0;
            cudaError_t e = hd == 128 ? attn_prepare_hd<128>(group, Hkv, cs, &clusters)
                                      : attn_prepare_hd<64>(group, Hkv, cs, &clusters);
            if (e != cudaSuccess) {
                cudaGetLastError();  // a cluster size the device refuses: try the next one
                continue;
            }
            if (clusters >= Hkv) best = cs;
        }
        if (!best) {
            best = cmax;
            LS_CK(hd == 128 ? attn_prepare_hd<128>(group, Hkv, best, nullptr) : attn_prepare_hd<64>(group, Hkv, best, nullptr));
        }
        AttnPlan p;
        p.csize = best;
        it = plans.emplace(key, p).first;
    }
    *out = it->second;
    return LS_OK;
}

// per-CTA argmax candidates the LM-head kernel of this family writes per row
int n_candidates(int path, int V, int K, int M)
{
    return path == LS_LINEAR_MMA ? mma_grid(EPI_ARGMAX, V, K, M) : lin_grid(EPI_ARGMAX, V);
}

LinArgs lin_args(const uint16_t* w, const uint16_t* h, int M, int N, int K)
{
    LinArgs a;
    memset(&a, 0, sizeof(a));
    a.w0 = a.w1 = a.w2 = w;
    a.n0 = N;
    a.n1 = 0;
    a.h = h;
    a.M = M;
    a.N = N;
    a.K = K;
    a.nseq = 1;
    return a;
}

// layers [l0, l1) on M residual rows starting at xrow; row r sits at ctl.cache_len + pos_off + r
// fused-RMSNorm fields of a consumer (sums it reads, sums it clears for the producer after
// it) and of a residual producer (sums it adds to, rows x*gain it leaves)
void norm_in(const ls_model* m, LinArgs& a, const long long* sums, long long* clear)
{
    a.ss_in = sums;
    a.ss_clear = clear;
    a.inv_d = 1.0f / (float)m->c.d_model;
    a.eps = m->c.rms_eps;
}
void norm_out(LinArgs& a, long long* sums, const uint16_t* gain_a, uint16_t* hout_a, const uint16_t* gain_b,
              uint16_t* hout_b)
{
    a.ss_out = sums;
    a.gain_a = gain_a;
    a.hout_a = gain_a ? hout_a : nullptr;
    a.gain_b = gain_b;
    a.hout_b = gain_b ? hout_b : nullptr;
}

// Layers [l0, l1) on M residual rows starting at xrow (row slot `slot` of the 16-row buffers);
// row r sits at ctl.cache_len + pos_off + r.  h_first: the rows x*gain for layer l0's first
// norm (left by the embedding, by the previous layer, or by a draft pass for the verify
// pass).  The last layer's down-projection leaves x*gain_end_a in the h rows (for the LM
// head or the next call) and x*gain_end_b in the exit-activation rows.
int run_layers(ls_model* m, int l0, int l1, int M, float* xrow, int pos_off, int slot, const uint16_t* h_first,
               const uint16_t* gain_end_a, const uint16_t* gain_end_b)
{
    const ls_config& c = m->c;
    const int D = c.d_model, Hq = c.n_heads, Hkv = c.n_kv_heads, hd = c.head_dim, F = c.d_ffn;
    const int qw = Hq * hd, kvw = Hkv * hd;
    const LaunchCtx st = {m->st, m->pdl};
    uint16_t* hrow = m->h + (size_t)slot * D;
    uint16_t* herow = m->hE + (size_t)slot * D;
    for (int l = l0; l < l1; ++l) {
        const LayerW& w = m->lw[l];
        uint16_t* kp = m->kpages + (size_t)l * m->layer_kv_elems;
        uint16_t* vp = m->vpages + (size_t)l * m->layer_kv_elems;
        LinArgs a = lin_args(w.wq, l == l0 ? h_first : hrow, M, qw + 2 * kvw, D);
        a.w1 = w.wk;
        a.w2 = w.wv;
        a.n0 = qw;
        a.n1 = kvw;
        a.ctl = m->ctl;
        a.inv_freq = m->inv_freq;
        a.page_table = m->pt;
        a.nseq = m->nseq;
        a.pt_stride = m->pt_stride;
        a.q_out = m->q;
        a.kpages = kp;
        a.vpages = vp;
        a.Hq = Hq;
        a.Hkv = Hkv;
        a.hd = hd;
        a.page_shift = m->page_shift;
        a.max_seq = m->seq_cap;
        a.pos_off = pos_off;
        a.theta = c.rope_theta;
        a.gate = m->gate;
        norm_in(m, a, m->ss_ffn + slot * kSsSlots, m->ss_attn + slot * kSsSlots);  // rows left by an embedding or a down projection
        LS_CK(launch_linear(m->path, EPI_QKV, a, st));
        LS_TRY(attn_launch(m->attn, m->q, kp, vp, m->pt, m->ctl, pos_off, M, Hq, Hkv, hd, m->page_shift, m->seq_cap, m->o,
                           st, m->gate, m->nseq, m->pt_stride));
        a = lin_args(w.wo, m->o, M, D, qw);
        a.out = xrow;
        a.ldo = D;
        a.ctl = m->ctl;
        a.gate = m->gate;
        norm_out(a, m->ss_attn + slot * kSsSlots, w.ffn_norm, hrow, nullptr, nullptr);
        LS_CK(launch_linear(m->path, EPI_RESIDUAL, a, st));
        a = lin_args(w.wg, hrow, M, F, D);
        a.w1 = w.wu;
        a.out_bf16 = m->a;
        a.ctl = m->ctl;
        a.gate = m->gate;
        norm_in(m, a, m->ss_attn + slot * kSsSlots, m->ss_ffn + slot * kSsSlots);
        LS_CK(launch_linear(m->path, EPI_SWIGLU, a, st));
        a = lin_args(w.wd, m->a, M, D, F);
        a.out = xrow;
        a.ldo = D;
        a.ctl = m->ctl;
        a.gate = m->gate;
        if (l + 1 < l1) norm_out(a, m->ss_ffn + slot * kSsSlots, m->lw[l + 1].attn_norm, hrow, nullptr, nullptr);
        else norm_out(a, m->ss_ffn + slot * kSsSlots, gain_end_a, hrow, gain_end_b, herow);
        LS_CK(launch_linear(m->path, EPI_RESIDUAL, a, st));
        m->launches += 5;
    }
    LS_CK(cudaGetLastError());
    return LS_OK;
}

// shared head g(.) = final norm + LM head (+ argmax) on the M rows of slot `slot`, whose
// x*final_gain rows and partial sums the last down-projection has left
// min_margin > 0 (the head of a draft pass, adaptive drafting): also reduce the second-largest
// logit and stop the step's drafting when the top-two margin falls below it
int run_head(ls_model* m, int M, int slot, int32_t* tok_out, float* logits, float min_margin = 0.f)
{
    const ls_config& c = m->c;
    const LaunchCtx st = {m->st, m->pdl};
    LinArgs a = lin_args(m->lm, m->h + (size_t)slot * c.d_model, M, c.vocab, c.d_model);
    a.cand = m->cand;
    a.cand_stride = m->cand_stride;
    a.out = logits;
    a.ldo = c.vocab;
    a.ctl = m->ctl;
    a.gate = m->gate;
    a.second = min_margin > 0.f ? m->second : nullptr;
    norm_in(m, a, m->ss_ffn + slot * kSsSlots, nullptr);
    LS_CK(launch_linear(m->path, EPI_ARGMAX, a, st));
    LS_CK(launch(st, argmax_finish_kernel, dim3(M), dim3(256), 0, (const ValIdx*)m->cand,
                 n_candidates(m->path, c.vocab, c.d_model, M), m->cand_stride, tok_out, m->ctl,
                 (const float*)a.second, min_margin, m->gate, m->next_pass));
    m->launches += 2;
    return LS_OK;
}

int run_embed(ls_model* m, const int32_t* tok_dev, int M, float* xrow, int slot, int tok_stride = 1)
{
    LS_CK(launch(LaunchCtx{m->st, m->pdl}, embed_kernel, dim3(M), dim3(256), 0, m->emb, tok_dev, m->c.d_model,
                 m->c.vocab, xrow, m->ctl, m->lw[0].attn_norm, m->h + (size_t)slot * m->c.d_model,
                 m->ss_ffn + slot * kSsSlots, m->gate, tok_stride));
    m->launches += 1;
    return LS_OK;
}

// ------------------------------------------------------------------ prompt pass (large M)
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn tensor_map_encoder()
{
    static TensorMapEncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (TensorMapEncodeFn)p;
    }
    return fn;
}

// 2-D map of a row-major bf16 matrix [rows, K]: boxes of 64 columns (128 bytes) x 128 rows,
// 128-byte swizzle, zeros outside the matrix
int make_tile_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t K, int box_rows)
{
    TensorMapEncodeFn fn = tensor_map_encoder();
    if (!fn) return LS_ERR_UNSUPPORTED;
    // A map depends on nothing but (address, extents, box): the prompt pass asks for the same few
    // hundred maps (every layer's weights, its own activation buffers) block after block, so they
    // are encoded once.  Bounded: the cache is dropped when it reaches 8192 entries.
    typedef std::tuple<const void*, uint64_t, uint64_t, int> MapKey;
    static std::map<MapKey, CUtensorMap> cache;
    static std::mutex mu;
    const MapKey key(ptr, rows, K, box_rows);
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = cache.find(key);
        if (it != cache.end()) {
            *map = it->second;
            return LS_OK;
        }
    }
    cuuint64_t dims[2] = {K, rows};
    cuuint64_t strides[1] = {K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kGemmBK, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return LS_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(mu);
    if (cache.size() >= 8192) cache.clear();
    cache.emplace(key, *map);
    return LS_OK;
}

// C[M, N] (+)= A[M, K] B[N, K]^T on the tensor cores (tcgen05), A and B bf16, C fp32
// more than one tile of rows: CTA pairs share each weight tile (a CTA stages half of it)
bool gemm_uses_pairs(int M)
{
    static const bool allowed = getenv("LS_NO_PAIR") == nullptr;
    return allowed && M > kGemmBM;
}

// C[M, n0 + n1 + n2] (+)= A[M, K] [B0; B1; B2]^T: up to three weight matrices with the same K
// in one launch (B1, B2 may be null).  swiglu_out (CTA pairs only; B0 = gate, B1 = up, n0 == n1):
// instead of C, bf16(silu(A B0^T) * (A B1^T)) [M, n0] is written.
int gemm_launch3(const uint16_t* A, const uint16_t* B0, int n0, const uint16_t* B1, int n1, const uint16_t* B2, int n2,
                 int M, int K, float* C, int ldc, int accumulate, int32_t* status, cudaStream_t st,
                 uint16_t* swiglu_out = nullptr, const RopeEpi* rope = nullptr)
{
    static bool allowed[64] = {false};
    int dev = 0;
    LS_CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !allowed[dev]) {
        LS_CK(cudaFuncSetAttribute(gemm_bf16_tn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmemBytes));
        if (dev >= 0 && dev < 64) allowed[dev] = true;
    }
    const bool pair = gemm_uses_pairs(M);
    CUtensorMap ma, mb[3];
    LS_TRY(make_tile_map(&ma, A, (uint64_t)M, (uint64_t)K, kGemmBM));
    const uint16_t* bs[3] = {B0, B1 ? B1 : B0, B2 ? B2 : B0};
    GemmSegs segs = {{n0, B1 ? n1 : 0, B2 ? n2 : 0}};
    int tiles = 0;
    for (int i = 0; i < 3; ++i) {
        const int rows = segs.n[i] > 0 ? segs.n[i] : n0;  // an unused slot still gets a valid map
        LS_TRY(make_tile_map(&mb[i], bs[i], (uint64_t)rows, (uint64_t)K, pair ? kGemmBN / 2 : kGemmBN));
        tiles += (segs.n[i] + kGemmBN - 1) / kGemmBN;
    }
    const int mtiles = (M + kGemmBM - 1) / kGemmBM;
    if (swiglu_out && !pair) return LS_ERR_INVALID_ARG;  // the fused epilogue exists on CTA pairs only
    if (swiglu_out) tiles = (n0 + kGemmBN / 2 - 1) / (kGemmBN / 2);
    if (pair) {
        // one CTA pair per two SMs, each walking its share of the 256 x 256 tiles
        static int max_pairs[64] = {0};
        cudaLaunchConfig_t cfg = {};
        cfg.stream = st;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = 2;
        at.val.clusterDim.y = 1;
        at.val.clusterDim.z = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        cfg.dynamicSmemBytes = kPairSmemBytes;
        cfg.blockDim = dim3(kPersistThreads);
        if (dev < 0 || dev >= 64) return LS_ERR_UNSUPPORTED;
        if (!max_pairs[dev]) {
            LS_CK(cudaFuncSetAttribute(gemm_bf16_tn_pair_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kPairSmemBytes));
            int sms = 0, n = 0;
            LS_CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
            cfg.gridDim = dim3(sms & ~1);
            LS_CK(cudaOccupancyMaxActiveClusters(&n, gemm_bf16_tn_pair_persistent_kernel, &cfg));
            if (n < 1) return LS_ERR_UNSUPPORTED;
            max_pairs[dev] = n < sms / 2 ? n : sms / 2;
        }
        const int n_tiles = tiles * ((mtiles + 1) / 2);
        const int pairs = n_tiles < max_pairs[dev] ? n_tiles : max_pairs[dev];
        cfg.gridDim = dim3(2 * pairs);
        RopeEpi re;
        memset(&re, 0, sizeof(re));
        if (rope) re = *rope;
        LS_CK(cudaLaunchKernelEx(&cfg, gemm_bf16_tn_pair_persistent_kernel, ma, mb[0], mb[1], mb[2], segs, M, K, C, ldc,
                                 accumulate, status, swiglu_out, re));
        return LS_OK;
    }
    if (rope) return LS_ERR_INVALID_ARG;  // the fused rotary epilogue exists on CTA pairs only
    dim3 grid(tiles, mtiles);
    gemm_bf16_tn_kernel<<<grid, 128, kGemmSmemBytes, st>>>(ma, mb[0], mb[1], mb[2], segs, M, K, C, ldc, accumulate, status);
    LS_CK(cudaGetLastError());
    return LS_OK;
}

int gemm_launch(const uint16_t* A, const uint16_t* B, int M, int N, int K, float* C, int ldc, int accumulate,
                int32_t* status, cudaStream_t st)
{
    return gemm_launch3(A, B, N, nullptr, 0, nullptr, 0, M, K, C, ldc, accumulate, status, st);
}

// cudaFuncAttributeMaxDynamicSharedMemorySize once per kernel and device (smem: the largest the kernel is launched with)
template <typename Kernel>
int allow_smem_once(Kernel kernel, size_t smem)
{
    static size_t allowed[64] = {0};
    int dev = 0;
    LS_CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || allowed[dev] < smem) {
        LS_CK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (dev >= 0 && dev < 64) allowed[dev] = smem;
    }
    return LS_OK;
}

// rows at positions pos0 .. pos0 + R - 1 over the paged cache of one layer (pool_pages pages).
// Head dim 128 and at least one full tile of rows: the tcgen05 kernel (status: where it reports a
// wait that ran out); otherwise the mma.sync walk (G <= 4) or the FMA walk.
bool attn_uses_tc(int R, int hd, int pos0, int page_shift)
{
    static const bool allowed = getenv("LS_NO_TC_ATTN") == nullptr && tensor_map_encoder() != nullptr;
    const int box_rows = (1 << page_shift) < kTcAttnKB ? (1 << page_shift) : kTcAttnKB;
    return allowed && hd == kTcAttnB && R >= kTcAttnB && (pos0 + R + box_rows - 1) / box_rows <= kTcAttnMaxBoxes;
}

int prefill_attn_launch(const uint16_t* q, const uint16_t* kp, const uint16_t* vp, const int32_t* pt, int pos0, int R,
                        int Hq, int Hkv, int hd, int page_shift, int pool_pages, uint16_t* out, int32_t* status,
                        cudaStream_t st)
{
    if (attn_uses_tc(R, hd, pos0, page_shift)) {
        const int ps = 1 << page_shift, box_rows = ps < kTcAttnKB ? ps : kTcAttnKB;
        CUtensorMap mq, mk, mv;
        LS_TRY(make_tile_map(&mq, q, (uint64_t)R, (uint64_t)Hq * hd, kTcAttnB));
        LS_TRY(make_tile_map(&mk, kp, (uint64_t)pool_pages * Hkv * ps, (uint64_t)hd, box_rows));
        LS_TRY(make_tile_map(&mv, vp, (uint64_t)pool_pages * Hkv * ps, (uint64_t)hd, box_rows));
        LS_TRY(allow_smem_once(prefill_attn_tc_kernel, kTcAttnSmemBytes));
        dim3 tgrid(Hq, (R + kTcAttnB - 1) / kTcAttnB);
        prefill_attn_tc_kernel<<<tgrid, kTcAttnThreads, kTcAttnSmemBytes, st>>>(mq, mk, mv, pt, pos0, R, Hq, Hkv, page_shift,
                                                                               box_rows, out, status);
        LS_CK(cudaGetLastError());
        return LS_OK;
    }
    const int G = Hq / Hkv, Q = G * kMaxRows;
    dim3 grid((R + 15) / 16, Hkv);
    if (G == 1 || G == 2 || G == 4) {  // tensor-core kernel: 64 queries per CTA, 16 per warp
        const int rpc = 64 / G;
        dim3 mgrid((R + rpc - 1) / rpc, Hkv);
        if (hd == 128) {
            const size_t sm = prefill_attn_fa_smem_bytes<128>();
            LS_TRY(allow_smem_once(prefill_attn_fa_kernel<128>, sm));
            prefill_attn_fa_kernel<128><<<mgrid, kFaThreads, sm, st>>>(q, kp, vp, pt, pos0, R, Hq, Hkv, page_shift, out);
        } else {
            const size_t sm = prefill_attn_fa_smem_bytes<64>();
            LS_TRY(allow_smem_once(prefill_attn_fa_kernel<64>, sm));
            prefill_attn_fa_kernel<64><<<mgrid, kFaThreads, sm, st>>>(q, kp, vp, pt, pos0, R, Hq, Hkv, page_shift, out);
        }
    } else if (hd == 128) {
        const size_t sm = prefill_attn_smem_bytes<128>(Q);
        LS_TRY(allow_smem_once(prefill_attn_kernel<128>, sm));
        prefill_attn_kernel<128><<<grid, kAttnThreads, sm, st>>>(q, kp, vp, pt, pos0, R, Hq, Hkv, page_shift, out);
    } else {
        const size_t sm = prefill_attn_smem_bytes<64>(Q);
        LS_TRY(allow_smem_once(prefill_attn_kernel<64>, sm));
        prefill_attn_kernel<64><<<grid, kAttnThreads, sm, st>>>(q, kp, vp, pt, pos0, R, Hq, Hkv, page_shift, out);
    }
    LS_CK(cudaGetLastError());
    return LS_OK;
}

// rows [r0, r0 + R) of the prompt (ids already on the device) through layers [0, layers):
// fills the KV cache of those positions.  Unfused on purpose: this pass is compute-bound.
int prefill_block(ls_model* m, int r0, int R, int layers)
{
    const ls_config& c = m->c;
    const int D = c.d_model, Hq = c.n_heads, Hkv = c.n_kv_heads, hd = c.head_dim, F = c.d_ffn;
    const int qw = Hq * hd, kvw = Hkv * hd, qkvw = qw + 2 * kvw;
    cudaStream_t st = m->st;
    const LaunchCtx lc = {st, false};
    int32_t* status = m->ctl + CTL_STATUS;
    LS_CK(launch(lc, embed_kernel, dim3(R), dim3(256), 0, m->emb, m->ids + r0, D, c.vocab, m->px, m->ctl, nullptr,
                 nullptr, nullptr, 0, 1));
    m->launches += 1;
    for (int l = 0; l < layers; ++l) {
        const LayerW& w = m->lw[l];
        uint16_t* kp = m->kpages + (size_t)l * m->layer_kv_elems;
        uint16_t* vp = m->vpages + (size_t)l * m->layer_kv_elems;
        LS_CK(launch(lc, rmsnorm_kernel, dim3(R), dim3(256), 0, m->px, w.attn_norm, D, c.rms_eps, m->ph, nullptr));
        if (gemm_uses_pairs(R)) {  // q|k|v, rotary embedding and cache append in one kernel
            const RopeEpi re = {m->rope_tab, m->pt, m->pq, kp, vp, Hq, Hkv, hd, m->page_shift, m->seq_cap, r0};
            LS_TRY(gemm_launch3(m->ph, w.wq, qw, w.wk, kvw, w.wv, kvw, R, D, m->py, qkvw, 0, status, st, nullptr, &re));
        } else {
            LS_TRY(gemm_launch3(m->ph, w.wq, qw, w.wk, kvw, w.wv, kvw, R, D, m->py, qkvw, 0, status, st));
            rope_append_rows_kernel<<<R, 256, 0, st>>>(m->py, Hq, Hkv, hd, m->inv_freq, m->page_shift, m->pt, m->seq_cap, r0,
                                                      m->pq, kp, vp, status);
        }
        LS_TRY(prefill_attn_launch(m->pq, kp, vp, m->pt, r0, R, Hq, Hkv, hd, m->page_shift, m->n_pages, m->po, status, st));
        LS_TRY(gemm_launch(m->po, w.wo, R, D, qw, m->px, D, 1, status, st));
        LS_CK(launch(lc, rmsnorm_kernel, dim3(R), dim3(256), 0, m->px, w.ffn_norm, D, c.rms_eps, m->ph, nullptr));
        if (gemm_uses_pairs(R)) {  // gate, up and SwiGLU in one kernel
            LS_TRY(gemm_launch3(m->ph, w.wg, F, w.wu, F, nullptr, 0, R, D, m->py, 2 * F, 0, status, st, m->pa));
        } else {
            LS_TRY(gemm_launch3(m->ph, w.wg, F, w.wu, F, nullptr, 0, R, D, m->py, 2 * F, 0, status, st));
            swiglu_rows_kernel<<<R, 256, 0, st>>>(m->py, F, m->pa);
        }
        LS_TRY(gemm_launch(m->pa, w.wd, R, D, F, m->px, D, 1, status, st));
        m->launches += gemm_uses_pairs(R) ? 7 : 9;  // pairs: rotary epilogue and SwiGLU live in the GEMMs
    }
    LS_CK(cudaGetLastError());
    return LS_OK;
}

// one step of the loop.  E == L with d == 0: plain greedy; E < L with d == 0: early exit.
// min_margin > 0: adaptive drafting.  Draft pass j (j >= 1) is enqueued with gate j, so it idles
// once an earlier pass's head has found its two largest exit logits closer than min_margin;
// the verify pass always runs on d + 1 rows (the rows beyond the kept drafts are stale and
// never read by the rows that count: causal attention, one dot product per output element).
// draft pass j of a step (j == d: the extra early pass, no head)
int enqueue_draft_pass(ls_model* m, int E, int d, int j, bool reuse, float min_margin)
{
    const int D = m->c.d_model, B = m->nseq;
    float* xr = m->x + (size_t)j * B * D;  // rows j B .. j B + B - 1: draft position j of every sequence
    m->gate = min_margin > 0.f ? j : 0;
    if (j == 0) LS_TRY(run_embed(m, m->ctl + CTL_CUR_TOK, B, xr, 0, CTL_WORDS));
    else LS_TRY(run_embed(m, m->draft + (size_t)(j - 1) * B, B, xr, j * B));
    // the exit-layer row goes to the LM head (final gain) and, pre-scaled by layer E's
    // gain, to the verify pass (the exit-layer cache of Sec. 4.3.3)
    LS_TRY(run_layers(m, 0, E, B, xr, j, j * B, m->h + (size_t)j * B * D, j < d ? m->fnorm : nullptr,
                      reuse ? m->lw[E].attn_norm : nullptr));
    if (j < d) LS_TRY(run_head(m, B, j * B, m->draft + (size_t)j * B, nullptr, min_margin));
    m->gate = 0;
    return LS_OK;
}

int enqueue_accept(ls_model* m, int d, bool adaptive)
{
    const LaunchCtx lc = {m->st, m->pdl};
    if (m->nseq > 1)
        LS_CK(launch(lc, accept_batch_kernel, dim3(1), dim3(32), 0, (const int32_t*)m->draft, (const int32_t*)m->verified, d,
                     m->nseq, m->ctl, m->out_ids, m->accepted, m->seq_cap));
    else
        LS_CK(launch(lc, accept_kernel, dim3(1), dim3(32), 0, (const int32_t*)m->draft, (const int32_t*)m->verified, d,
                     m->ctl, m->out_ids, m->accepted, adaptive ? 1 : 0, adaptive ? m->drafted : (int32_t*)nullptr));
    m->launches += 1;
    return LS_OK;
}

// verify pass + accept of a step
int enqueue_verify(ls_model* m, int E, int d, bool reuse, float min_margin)
{
    const int D = m->c.d_model, L = m->c.n_layers, B = m->nseq;
    if (reuse) {
        // self-verification (Sec. 4.3.2) from the exit-layer activations
        LS_TRY(run_layers(m, E, L, (d + 1) * B, m->x, 0, 0, m->hE, m->fnorm, nullptr));
    } else {
        // the ablation of Sec. 7 (Table 7): no exit-layer cache, verification recomputes the
        // early layers of all d+1 rows (and rewrites their k, v with the same values)
        LS_TRY(run_embed(m, m->ctl + CTL_CUR_TOK, B, m->x, 0, CTL_WORDS));
        LS_TRY(run_embed(m, m->draft, d * B, m->x + (size_t)B * D, B));
        LS_TRY(run_layers(m, 0, L, (d + 1) * B, m->x, 0, 0, m->h, m->fnorm, nullptr));
    }
    LS_TRY(run_head(m, (d + 1) * B, 0, m->verified, nullptr));
    return enqueue_accept(m, d, min_margin > 0.f);
}

int enqueue_step(ls_model* m, int E, int d, bool reuse, float min_margin = 0.f)
{
    if (d == 0) {
        LS_TRY(run_embed(m, m->ctl + CTL_CUR_TOK, m->nseq, m->x, 0, CTL_WORDS));
        LS_TRY(run_layers(m, 0, E, m->nseq, m->x, 0, 0, m->h, m->fnorm, nullptr));
        LS_TRY(run_head(m, m->nseq, 0, m->verified, nullptr));
        return enqueue_accept(m, 0, false);
    }
    for (int j = 0; j <= (reuse ? d : d - 1); ++j)  // self-drafting (Sec. 4.3.1) + the extra early pass
        LS_TRY(enqueue_draft_pass(m, E, d, j, reuse, min_margin));
    return enqueue_verify(m, E, d, reuse, min_margin);
}

// The adaptive step as a graph whose draft passes 1..d are conditional (IF) nodes: the head of
// pass j - 1 switches pass j on when it keeps its draft, so a step that stops drafting early
// launches nothing for the passes it skips (as plain kernel nodes they would each still
// cost their ~40 launches).  The handles fall back to "off" at every launch of the graph.
int capture_adaptive_step(ls_model* m, int E, int d, float min_margin, cudaGraph_t* out)
{
    cudaGraph_t graph = nullptr;
    LS_CK(cudaGraphCreate(&graph, 0));
    cudaStream_t side = nullptr;
    cudaStream_t mainst = m->st;
    auto fail = [&](int rc) {
        m->st = mainst;
        m->next_pass = 0;
        if (side) cudaStreamDestroy(side);
        cudaGraphDestroy(graph);
        return rc;
    };
    std::vector<cudaGraphConditionalHandle> on(d + 1, 0);
    for (int j = 1; j <= d; ++j)
        if (cudaGraphConditionalHandleCreate(&on[j], graph, 0, cudaGraphCondAssignDefault) != cudaSuccess)
            return fail(LS_ERR_CUDA);
    if (cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking) != cudaSuccess) return fail(LS_ERR_CUDA);
    if (cudaStreamBeginCaptureToGraph(mainst, graph, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed) != cudaSuccess)
        return fail(LS_ERR_CUDA);
    auto abort_capture = [&](int rc) {
        cudaGraph_t g = nullptr;
        cudaStreamEndCapture(mainst, &g);
        return fail(rc);
    };
    m->next_pass = on[1];
    int rc = enqueue_draft_pass(m, E, d, 0, true, min_margin);
    if (rc != LS_OK) return abort_capture(rc);
    for (int j = 1; j <= d; ++j) {
        cudaStreamCaptureStatus status;
        cudaGraph_t cg = nullptr;
        const cudaGraphNode_t* deps = nullptr;
        size_t n_deps = 0;
        if (cudaStreamGetCaptureInfo(mainst, &status, nullptr, &cg, &deps, &n_deps) != cudaSuccess)
            return abort_capture(LS_ERR_CUDA);
        cudaGraphNodeParams p = {};
        p.type = cudaGraphNodeTypeConditional;
        p.conditional.handle = on[j];
        p.conditional.type = cudaGraphCondTypeIf;
        p.conditional.size = 1;
        cudaGraphNode_t node;
        if (cudaGraphAddNode(&node, graph, deps, n_deps, &p) != cudaSuccess) return abort_capture(LS_ERR_CUDA);
        if (cudaStreamUpdateCaptureDependencies(mainst, &node, 1, cudaStreamSetCaptureDependencies) != cudaSuccess)
            return abort_capture(LS_ERR_CUDA);
        cudaGraph_t body = p.conditional.phGraph_out[0];
        if (cudaStreamBeginCaptureToGraph(side, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed) != cudaSuccess)
            return abort_capture(LS_ERR_CUDA);
        m->st = side;
        m->next_pass = j < d ? on[j + 1] : 0;
        rc = enqueue_draft_pass(m, E, d, j, true, min_margin);
        m->st = mainst;
        cudaGraph_t captured = nullptr;
        cudaError_t e = cudaStreamEndCapture(side, &captured);
        if (rc != LS_OK) return abort_capture(rc);
        if (e != cudaSuccess) {
            g_last_cuda = (int)e;
            return abort_capture(LS_ERR_CUDA);
        }
    }
    m->next_pass = 0;
    rc = enqueue_verify(m, E, d, true, min_margin);
    cudaGraph_t done = nullptr;
    cudaError_t e = cudaStreamEndCapture(mainst, &done);
    if (rc != LS_OK) return fail(rc);
    if (e != cudaSuccess) {
        g_last_cuda = (int)e;
        return fail(LS_ERR_CUDA);
    }
    cudaStreamDestroy(side);
    *out = graph;
    return LS_OK;
}

void drop_graphs(ls_model* m)
{
    for (auto& kv : m->graphs) cudaGraphExecDestroy(kv.second.exec);
    m->graphs.clear();
}

int get_graph(ls_model* m, int E, int d, bool reuse, float min_margin, ls_model::G** out)
{
    uint32_t mbits;
    memcpy(&mbits, &min_margin, sizeof(mbits));
    const std::pair<uint64_t, uint32_t> key(
        ((uint64_t)m->nseq << 52) | ((uint64_t)(reuse ? 0 : 1) << 48) | ((uint64_t)E << 32) | ((uint64_t)d << 16), mbits);
    auto it = m->graphs.find(key);
    if (it == m->graphs.end()) {
        if (m->graphs.size() >= 64) drop_graphs(m);  // a bound on what a long-lived handle keeps
        cudaGraph_t graph = nullptr;
        int64_t before = m->launches;
        cudaError_t e = cudaSuccess;
        if (min_margin > 0.f && reuse && d > 0 && m->cond_graphs) {
            // a driver without conditional nodes (or out of handles): from now on the adaptive
            // step is the ordinary capture, whose skipped draft passes idle on their gate
            if (capture_adaptive_step(m, E, d, min_margin, &graph) != LS_OK) {
                cudaGetLastError();
                m->cond_graphs = false;
                m->launches = before;
                graph = nullptr;
            }
        }
        if (!graph) {
            LS_CK(cudaStreamBeginCapture(m->st, cudaStreamCaptureModeRelaxed));
            int rc = enqueue_step(m, E, d, reuse, min_margin);
            e = cudaStreamEndCapture(m->st, &graph);
            if (rc != LS_OK) {
                if (graph) cudaGraphDestroy(graph);
                return rc;
            }
            LS_CK(e);
        }
        ls_model::G g;
        g.nodes = m->launches - before;
        e = cudaGraphInstantiate(&g.exec, graph, 0);
        cudaGraphDestroy(graph);
        LS_CK(e);
        it = m->graphs.emplace(key, g).first;
    }
    *out = &it->second;
    return LS_OK;
}

int write_ctl(ls_model* m, int cache_len, int cur, int max_new)
{
    int32_t w[CTL_WORDS] = {cache_len, cur, 0, 0, 0, max_new, m->c.eos_id, 0, kNoStop};
    LS_CK(cudaMemcpyAsync(m->ctl, w, sizeof(w), cudaMemcpyHostToDevice, m->st));
    LS_CK(cudaStreamSynchronize(m->st));  // w is a stack array
    return LS_OK;
}

int read_ctl(ls_model* m, int32_t* w)
{
    LS_CK(cudaMemcpyAsync(w, m->ctl, sizeof(int32_t) * CTL_WORDS, cudaMemcpyDeviceToHost, m->st));
    LS_CK(cudaStreamSynchronize(m->st));
    return LS_OK;
}

int check_ids(const ls_model* m, const int32_t* ids, int n)
{
    if (!ids || n < 1) return LS_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= m->c.vocab) return LS_ERR_INVALID_ARG;
    return LS_OK;
}

// rows 0 .. n_prompt-2 of one prompt through `layers` layers into the cache of the sequence the
// model's view (pt, seq_cap) points at; the last prompt token is the first input of the loop
int prefill_rows(ls_model* m, const int32_t* prompt, int n_prompt, int layers)
{
    LS_CK(cudaMemcpyAsync(m->ids, prompt, sizeof(int32_t) * n_prompt, cudaMemcpyHostToDevice, m->st));
    LS_TRY(write_ctl(m, 0, 0, 0));
    const int rows = n_prompt - 1;
    if (rows > kMaxRows && m->big_prefill) {
        // the prompt pass proper: blocks of up to 1024 rows on the tensor cores
        const int pb = m->c.max_seq < kPrefillBlock ? m->c.max_seq : kPrefillBlock;
        for (int r0 = 0; r0 < rows; r0 += pb) LS_TRY(prefill_block(m, r0, rows - r0 < pb ? rows - r0 : pb, layers));
    } else {
        for (int r0 = 0; r0 < rows; r0 += kMaxRows) {
            int M = rows - r0;
            if (M > kMaxRows) M = kMaxRows;
            LS_TRY(run_embed(m, m->ids + r0, M, m->x, 0));
            LS_TRY(run_layers(m, 0, layers, M, m->x, r0, 0, m->h, nullptr, nullptr));
        }
    }
    return LS_OK;
}

// the model's view of its sequences for the duration of a call
struct SeqView {
    ls_model* m;
    SeqView(ls_model* m_, int nseq, int pt_stride, int cap, const int32_t* pt) : m(m_)
    {
        m->nseq = nseq;
        m->pt_stride = pt_stride;
        m->seq_cap = cap;
        m->pt = pt;
    }
    ~SeqView()
    {
        m->nseq = 1;
        m->pt_stride = 0;
        m->seq_cap = m->c.max_seq;
        m->pt = m->page_table;
    }
};

// algorithmic bytes of one sequence's schedule: weights of `steps` steps and the k, v rows read
void schedule_bytes(const ls_config& c, int E, int d, bool reuse, int n_prompt, const int32_t* acc, const int32_t* kept,
                    int steps, int64_t* wb_out, int64_t* kb_out, int64_t* acc_out)
{
    const int L = c.n_layers;
    const int64_t qw = (int64_t)c.n_heads * c.head_dim, kvw = (int64_t)c.n_kv_heads * c.head_dim;
    const int64_t w_layer = 2 * ((qw + 2 * kvw) * c.d_model + qw * c.d_model + 3 * (int64_t)c.d_model * c.d_ffn);
    const int64_t w_lm = 2 * (int64_t)c.vocab * c.d_model;
    const int64_t kvb = 2 * 2 * kvw;
    int64_t wb = 0, kb = 0, cl = n_prompt - 1, acc_sum = 0;
    for (int s = 0; s < steps; ++s) {
        const int n = acc[s];
        if (d == 0) {
            wb += E * w_layer + w_lm;
            kb += (int64_t)E * kvb * (cl + 1);
        } else if (reuse) {
            // draft passes that ran: all d + 1, or with an early stop the k + 1 up to the one
            // whose head stopped the drafting (k drafts kept); heads: one per pass but the extra one
            const int k = kept ? kept[s] : d;
            const int heads = k < d ? k + 1 : d;
            wb += (int64_t)(k + 1) * E * w_layer + (int64_t)heads * w_lm + (int64_t)(L - E) * w_layer + w_lm;
            for (int j = 0; j <= k; ++j) kb += (int64_t)E * kvb * (cl + j + 1);
            kb += (int64_t)(L - E) * kvb * (cl + k + 1);
        } else {
            wb += (int64_t)d * (E * w_layer + w_lm) + (int64_t)L * w_layer + w_lm;
            for (int j = 0; j < d; ++j) kb += (int64_t)E * kvb * (cl + j + 1);
            kb += (int64_t)L * kvb * (cl + d + 1);
        }
        cl += n + 1;
        acc_sum += n;
    }
    *wb_out = wb;
    *kb_out = kb;
    *acc_out = acc_sum;
}

int decode_loop(ls_model* m, int32_t exit_layer, int32_t num_draft, int32_t max_new, int32_t flags, float min_margin);

}  // namespace

// =============================================================================== C ABI
extern "C" {

const char* ls_strerror(int s)
{
    switch (s) {
        case LS_OK: return "ok";
        case LS_ERR_INVALID_ARG: return "invalid argument";
        case LS_ERR_CAPACITY: return "capacity exceeded (KV cache, workspace or max_draft)";
        case LS_ERR_CUDA: return "CUDA runtime error (see ls_last_cuda_error)";
        case LS_ERR_DEVICE_STATUS: return "a kernel's bounds check refused an access";
        case LS_ERR_UNSUPPORTED: return "unsupported device or shape";
        default: return "unknown status";
    }
}

int ls_last_cuda_error(void) { return g_last_cuda; }

size_t ls_workspace_bytes(const ls_config* cfg)
{
    if (!config_ok(cfg)) return 0;
    return carve(*cfg, nullptr, nullptr);
}

int ls_model_create(const ls_config* cfg, const ls_weights* w, void* workspace, size_t workspace_bytes,
                    void* cuda_stream, ls_model** out)
{
    if (!out) return LS_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg) || !w || !workspace) return LS_ERR_INVALID_ARG;
    if (((uintptr_t)workspace & 255u) != 0) return LS_ERR_INVALID_ARG;
    if (workspace_bytes < carve(*cfg, nullptr, nullptr)) return LS_ERR_CAPACITY;
    int dev = 0;
    cudaDeviceProp prop;
    LS_CK(cudaGetDevice(&dev));
    LS_CK(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return LS_ERR_UNSUPPORTED;
    if (!aligned16(w->tok_embed) || !aligned16(w->final_norm) || !aligned16(w->lm_head)) return LS_ERR_INVALID_ARG;
    const void* const* per[9] = {w->attn_norm, w->wq, w->wk, w->wv, w->wo, w->ffn_norm, w->w_gate, w->w_up, w->w_down};
    for (int i = 0; i < 9; ++i) {
        if (!per[i]) return LS_ERR_INVALID_ARG;
        for (int l = 0; l < cfg->n_layers; ++l)
            if (!aligned16(per[i][l])) return LS_ERR_INVALID_ARG;
    }
    ls_model* m = new (std::nothrow) ls_model();
    if (!m) return LS_ERR_CAPACITY;
    m->c = *cfg;
    m->path = cfg->linear_path == LS_LINEAR_AUTO ? (cfg->max_draft + 1 > 4 ? LS_LINEAR_MMA : LS_LINEAR_FMA)
                                                 : cfg->linear_path;
    if (const char* e = getenv("LS_LINEAR_PATH")) {
        if (!strcmp(e, "fma")) m->path = LS_LINEAR_FMA;
        if (!strcmp(e, "mma")) m->path = LS_LINEAR_MMA;
    }
    m->st = (cudaStream_t)cuda_stream;
    m->own_stream = false;
    if (!m->st) {
        // the legacy default stream cannot be captured into a graph: use a stream of our own
        // (a blocking one, so that it still orders after the caller's default-stream work)
        cudaError_t se = cudaStreamCreate(&m->st);
        if (se != cudaSuccess) {
            g_last_cuda = (int)se;
            delete m;
            return LS_ERR_CUDA;
        }
        m->own_stream = true;
    }
    m->emb = (const uint16_t*)w->tok_embed;
    m->fnorm = (const uint16_t*)w->final_norm;
    m->lm = (const uint16_t*)w->lm_head;
    m->lw.resize(cfg->n_layers);
    for (int l = 0; l < cfg->n_layers; ++l) {
        LayerW& x = m->lw[l];
        x.attn_norm = (const uint16_t*)w->attn_norm[l];
        x.wq = (const uint16_t*)w->wq[l];
        x.wk = (const uint16_t*)w->wk[l];
        x.wv = (const uint16_t*)w->wv[l];
        x.wo = (const uint16_t*)w->wo[l];
        x.ffn_norm = (const uint16_t*)w->ffn_norm[l];
        x.wg = (const uint16_t*)w->w_gate[l];
        x.wu = (const uint16_t*)w->w_up[l];
        x.wd = (const uint16_t*)w->w_down[l];
    }
    size_t used = carve(*cfg, (unsigned char*)workspace, m);
    m->n_prompt = 0;
    m->prefilled_layers = 0;
    m->nseq = 1;
    m->pt_stride = 0;
    m->seq_cap = cfg->max_seq;
    m->pt = m->page_table;
    m->use_graphs = getenv("LS_NO_GRAPH") == nullptr;
    m->pdl = getenv("LS_NO_PDL") == nullptr;
    m->cond_graphs = getenv("LS_NO_COND") == nullptr;
    m->gate = 0;
    m->next_pass = 0;
    m->big_prefill = getenv("LS_SMALL_PREFILL") == nullptr && tensor_map_encoder() != nullptr;
    m->launches = 0;
    memset(&m->stats, 0, sizeof(m->stats));
    m->h_n_out = m->h_n_steps = 0;
    m->ev0 = m->ev1 = nullptr;
    auto fail = [&](int rc) {
        if (m->ev0) cudaEventDestroy(m->ev0);
        if (m->ev1) cudaEventDestroy(m->ev1);
        if (m->own_stream) cudaStreamDestroy(m->st);
        delete m;
        return rc;
    };
    cudaError_t e = cudaMemsetAsync(workspace, 0, used, m->st);
    if (e == cudaSuccess) {
        std::vector<int32_t> pt(m->n_pages);
        for (int i = 0; i < m->n_pages; ++i) pt[i] = i;
        std::vector<float> fr(cfg->head_dim / 2);
        for (int j = 0; j < cfg->head_dim / 2; ++j)
            fr[j] = (float)pow((double)cfg->rope_theta, -2.0 * (double)j / (double)cfg->head_dim);
        e = cudaMemcpyAsync(m->page_table, pt.data(), sizeof(int32_t) * pt.size(), cudaMemcpyHostToDevice, m->st);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(m->inv_freq, fr.data(), sizeof(float) * fr.size(), cudaMemcpyHostToDevice, m->st);
        if (e == cudaSuccess) {
            rope_table_kernel<<<cfg->max_seq, cfg->head_dim / 2, 0, m->st>>>(m->inv_freq, cfg->head_dim / 2, m->rope_tab);
            e = cudaGetLastError();
        }
        if (e == cudaSuccess) e = cudaStreamSynchronize(m->st);
    }
    if (e == cudaSuccess) e = cudaEventCreate(&m->ev0);
    if (e == cudaSuccess) e = cudaEventCreate(&m->ev1);
    if (e != cudaSuccess) {
        g_last_cuda = (int)e;
        return fail(LS_ERR_CUDA);
    }
    int rc = attn_plan(cfg->head_dim, cfg->n_heads / cfg->n_kv_heads, cfg->n_kv_heads, cfg->max_seq, &m->attn);
    if (rc != LS_OK) return fail(rc);
    *out = m;
    return LS_OK;
}

int ls_model_destroy(ls_model* m)
{
    if (!m) return LS_ERR_INVALID_ARG;
    cudaStreamSynchronize(m->st);
    drop_graphs(m);
    cudaEventDestroy(m->ev0);
    cudaEventDestroy(m->ev1);
    if (m->own_stream) cudaStreamDestroy(m->st);
    delete m;
    return LS_OK;
}

int ls_set_page_table(ls_model* m, const int32_t* table, int32_t n_pages)
{
    if (!m || !table || n_pages != m->n_pages) return LS_ERR_INVALID_ARG;
    std::vector<char> seen(n_pages, 0);
    for (int i = 0; i < n_pages; ++i) {
        if (table[i] < 0 || table[i] >= n_pages || seen[table[i]]) return LS_ERR_INVALID_ARG;
        seen[table[i]] = 1;
    }
    LS_CK(cudaMemcpyAsync(m->page_table, table, sizeof(int32_t) * n_pages, cudaMemcpyHostToDevice, m->st));
    LS_CK(cudaStreamSynchronize(m->st));
    m->n_prompt = 0;  // cached positions moved
    return LS_OK;
}

int ls_prefill(ls_model* m, const int32_t* prompt, int32_t n_prompt, int32_t layers)
{
    if (!m) return LS_ERR_INVALID_ARG;
    LS_TRY(check_ids(m, prompt, n_prompt));
    const int L = m->c.n_layers;
    if (layers == 0) layers = L;
    if (layers < 1 || layers > L) return LS_ERR_INVALID_ARG;
    if (n_prompt > m->c.max_seq) return LS_ERR_CAPACITY;
    m->n_prompt = 0;
    m->b_n_prompt.clear();
    LS_CK(cudaEventRecord(m->ev0, m->st));
    LS_TRY(prefill_rows(m, prompt, n_prompt, layers));
    LS_CK(cudaEventRecord(m->ev1, m->st));
    int32_t w[CTL_WORDS];
    LS_TRY(read_ctl(m, w));
    if (w[CTL_STATUS]) return LS_ERR_DEVICE_STATUS;
    float ms = 0.f;
    LS_CK(cudaEventElapsedTime(&ms, m->ev0, m->ev1));
    m->stats.prefill_ms = ms;
    m->n_prompt = n_prompt;
    m->last_tok = prompt[n_prompt - 1];
    m->prefilled_layers = layers;
    return LS_OK;
}

int ls_decode(ls_model* m, int32_t exit_layer, int32_t num_draft, int32_t max_new)
{
    return ls_decode_flags(m, exit_layer, num_draft, max_new, 0);
}

int ls_decode_flags(ls_model* m, int32_t exit_layer, int32_t num_draft, int32_t max_new, int32_t flags)
{
    return decode_loop(m, exit_layer, num_draft, max_new, flags, 0.f);
}

int ls_decode_adaptive(ls_model* m, int32_t exit_layer, int32_t max_draft, float min_margin, int32_t max_new)
{
    if (!(min_margin > 0.f)) return LS_ERR_INVALID_ARG;  // also refuses NaN
    if (exit_layer < 1 || max_draft < 1) return LS_ERR_INVALID_ARG;
    return decode_loop(m, exit_layer, max_draft, max_new, 0, min_margin);
}

}  // extern "C"

namespace {
int decode_loop(ls_model* m, int32_t exit_layer, int32_t num_draft, int32_t max_new, int32_t flags, float min_margin)
{
    if (!m || m->n_prompt < 1 || (flags & ~LS_DECODE_NO_EXIT_CACHE)) return LS_ERR_INVALID_ARG;
    const bool reuse = !(flags & LS_DECODE_NO_EXIT_CACHE);
    const bool adaptive = min_margin > 0.f;
    const ls_config& c = m->c;
    const int L = c.n_layers;
    int E = exit_layer, d = num_draft;
    if (max_new < 1 || d < 0 || E < 0) return LS_ERR_INVALID_ARG;
    if (E == 0) {
        if (d != 0) return LS_ERR_INVALID_ARG;
        E = L;  // plain greedy
    } else if (d == 0) {
        if (E > L) return LS_ERR_INVALID_ARG;  // early exit
    } else {
        if (E > L - 1) return LS_ERR_INVALID_ARG;
        if (d > c.max_draft) return LS_ERR_CAPACITY;
    }
    const int need_layers = (d > 0) ? L : E;
    if (m->prefilled_layers < need_layers) return LS_ERR_INVALID_ARG;
    if ((int64_t)m->n_prompt + max_new + d + 1 > c.max_seq) return LS_ERR_CAPACITY;

    ls_model::G* g = nullptr;
    if (m->use_graphs) LS_TRY(get_graph(m, E, d, reuse, min_margin, &g));
    LS_TRY(write_ctl(m, m->n_prompt - 1, m->last_tok, max_new));
    int64_t launched = 0;
    int syncs = 0, n_out = 0, steps_done = 0;
    int32_t w[CTL_WORDS];
    LS_CK(cudaEventRecord(m->ev0, m->st));
    for (;;) {
        // first batch: as if every draft were accepted; afterwards at the observed rate
        int remaining = max_new - n_out;
        int steps = (remaining + d) / (d + 1);
        if (steps_done > 0 && n_out > 0) {
            int64_t est = ((int64_t)remaining * steps_done + n_out - 1) / n_out;
            steps = (int)(est < 1 ? 1 : est);
        }
        for (int i = 0; i < steps; ++i) {
            if (g) {
                LS_CK(cudaGraphLaunch(g->exec, m->st));
                launched += g->nodes;
            } else {
                int64_t before = m->launches;
                LS_TRY(enqueue_step(m, E, d, reuse, min_margin));
                launched += m->launches - before;
            }
        }
        LS_TRY(read_ctl(m, w));
        ++syncs;
        if (w[CTL_STATUS]) return LS_ERR_DEVICE_STATUS;
        n_out = w[CTL_N_OUT];
        steps_done = w[CTL_N_STEPS];
        if (w[CTL_DONE]) break;
    }
    LS_CK(cudaEventRecord(m->ev1, m->st));
    LS_CK(cudaEventSynchronize(m->ev1));
    float ms = 0.f;
    LS_CK(cudaEventElapsedTime(&ms, m->ev0, m->ev1));

    m->h_n_out = w[CTL_N_OUT];
    m->h_n_steps = w[CTL_N_STEPS];
    m->h_out.resize(m->h_n_out);
    m->h_acc.resize(m->h_n_steps);
    m->h_drafted.assign(m->h_n_steps, d);
    LS_CK(cudaMemcpyAsync(m->h_out.data(), m->out_ids, sizeof(int32_t) * m->h_n_out, cudaMemcpyDeviceToHost, m->st));
    LS_CK(cudaMemcpyAsync(m->h_acc.data(), m->accepted, sizeof(int32_t) * m->h_n_steps, cudaMemcpyDeviceToHost, m->st));
    if (adaptive)
        LS_CK(cudaMemcpyAsync(m->h_drafted.data(), m->drafted, sizeof(int32_t) * m->h_n_steps, cudaMemcpyDeviceToHost,
                              m->st));
    LS_CK(cudaStreamSynchronize(m->st));

    // algorithmic bytes of the schedule (matrices only; norm gains and activations are noise)
    int64_t wb = 0, kb = 0, acc_sum = 0;
    schedule_bytes(c, E, d, reuse, m->n_prompt, m->h_acc.data(), adaptive ? m->h_drafted.data() : nullptr, m->h_n_steps, &wb,
                   &kb, &acc_sum);
    m->stats.decode_ms = ms;
    m->stats.weight_bytes = wb;
    m->stats.kv_bytes = kb;
    m->stats.kernel_launches = launched;
    m->stats.n_generated = m->h_n_out;
    m->stats.n_steps = m->h_n_steps;
    m->stats.n_accepted = (int32_t)acc_sum;
    m->stats.host_syncs = syncs;
    return LS_OK;
}
}  // namespace

extern "C" {

int ls_read_drafted(ls_model* m, int32_t* drafted, int32_t* out_steps)
{
    if (!m) return LS_ERR_INVALID_ARG;
    if (drafted && m->h_n_steps) memcpy(drafted, m->h_drafted.data(), sizeof(int32_t) * m->h_n_steps);
    if (out_steps) *out_steps = m->h_n_steps;
    return LS_OK;
}

int ls_read_output(ls_model* m, int32_t* out_ids, int32_t* out_n, int32_t* accepted, int32_t* out_steps)
{
    if (!m) return LS_ERR_INVALID_ARG;
    if (out_ids && m->h_n_out) memcpy(out_ids, m->h_out.data(), sizeof(int32_t) * m->h_n_out);
    if (out_n) *out_n = m->h_n_out;
    if (accepted && m->h_n_steps) memcpy(accepted, m->h_acc.data(), sizeof(int32_t) * m->h_n_steps);
    if (out_steps) *out_steps = m->h_n_steps;
    return LS_OK;
}

int ls_generate(ls_model* m, const int32_t* prompt, int32_t n_prompt, int32_t exit_layer, int32_t num_draft,
                int32_t max_new, int32_t* out_ids, int32_t* out_n, int32_t* accepted, int32_t* out_steps)
{
    if (!m || !out_ids || !out_n || !accepted || !out_steps) return LS_ERR_INVALID_ARG;
    if (exit_layer < 1 || exit_layer > m->c.n_layers - 1 || num_draft < 1 || max_new < 1) return LS_ERR_INVALID_ARG;
    if (num_draft > m->c.max_draft) return LS_ERR_CAPACITY;
    if (n_prompt < 1) return LS_ERR_INVALID_ARG;
    if ((int64_t)n_prompt + max_new + num_draft + 1 > m->c.max_seq) return LS_ERR_CAPACITY;
    LS_TRY(ls_prefill(m, prompt, n_prompt, 0));
    LS_TRY(ls_decode(m, exit_layer, num_draft, max_new));
    return ls_read_output(m, out_ids, out_n, accepted, out_steps);
}

int ls_generate_adaptive(ls_model* m, const int32_t* prompt, int32_t n_prompt, int32_t exit_layer, int32_t max_draft,
                         float min_margin, int32_t max_new, int32_t* out_ids, int32_t* out_n, int32_t* accepted,
                         int32_t* drafted, int32_t* out_steps)
{
    if (!m || !out_ids || !out_n || !accepted || !drafted || !out_steps) return LS_ERR_INVALID_ARG;
    if (exit_layer < 1 || exit_layer > m->c.n_layers - 1 || max_draft < 1 || max_new < 1) return LS_ERR_INVALID_ARG;
    if (!(min_margin > 0.f)) return LS_ERR_INVALID_ARG;
    if (max_draft > m->c.max_draft) return LS_ERR_CAPACITY;
    if (n_prompt < 1) return LS_ERR_INVALID_ARG;
    if ((int64_t)n_prompt + max_new + max_draft + 1 > m->c.max_seq) return LS_ERR_CAPACITY;
    LS_TRY(ls_prefill(m, prompt, n_prompt, 0));
    LS_TRY(ls_decode_adaptive(m, exit_layer, max_draft, min_margin, max_new));
    LS_TRY(ls_read_drafted(m, drafted, nullptr));
    return ls_read_output(m, out_ids, out_n, accepted, out_steps);
}

int ls_generate_full(ls_model* m, const int32_t* prompt, int32_t n_prompt, int32_t max_new, int32_t* out_ids,
                     int32_t* out_n)
{
    if (!m || !out_ids || !out_n || max_new < 1 || n_prompt < 1) return LS_ERR_INVALID_ARG;
    if ((int64_t)n_prompt + max_new + 1 > m->c.max_seq) return LS_ERR_CAPACITY;
    LS_TRY(ls_prefill(m, prompt, n_prompt, 0));
    LS_TRY(ls_decode(m, 0, 0, max_new));
    return ls_read_output(m, out_ids, out_n, nullptr, nullptr);
}

int ls_generate_early(ls_model* m, const int32_t* prompt, int32_t n_prompt, int32_t exit_layer, int32_t max_new,
                      int32_t* out_ids, int32_t* out_n)
{
    if (!m || !out_ids || !out_n || max_new < 1 || n_prompt < 1) return LS_ERR_INVALID_ARG;
    if (exit_layer < 1 || exit_layer > m->c.n_layers) return LS_ERR_INVALID_ARG;
    if ((int64_t)n_prompt + max_new + 1 > m->c.max_seq) return LS_ERR_CAPACITY;
    LS_TRY(ls_prefill(m, prompt, n_prompt, exit_layer));
    LS_TRY(ls_decode(m, exit_layer, 0, max_new));
    return ls_read_output(m, out_ids, out_n, nullptr, nullptr);
}

// ------------------------------------------------------------------ several sequences per pass
int ls_prefill_batch(ls_model* m, int32_t n_seq, const int32_t* prompts, const int32_t* prompt_lens)
{
    if (!m || !prompts || !prompt_lens || n_seq < 1 || n_seq > LS_MAX_ROWS) return LS_ERR_INVALID_ARG;
    const int pps = m->n_pages / n_seq, cap = pps * m->c.page_size;  // pages and positions per sequence
    size_t off = 0;
    for (int b = 0; b < n_seq; ++b) {
        LS_TRY(check_ids(m, prompts + off, prompt_lens[b]));
        if (prompt_lens[b] > cap) return LS_ERR_CAPACITY;
        off += prompt_lens[b];
    }
    m->n_prompt = 0;  // the single-sequence state is gone: the sequences share its pages
    m->b_n_prompt.clear();
    m->b_last_tok.clear();
    LS_CK(cudaEventRecord(m->ev0, m->st));
    off = 0;
    for (int b = 0; b < n_seq; ++b) {
        SeqView view(m, 1, 0, cap, m->page_table + (size_t)b * pps);
        LS_TRY(prefill_rows(m, prompts + off, prompt_lens[b], m->c.n_layers));
        off += prompt_lens[b];
    }
    LS_CK(cudaEventRecord(m->ev1, m->st));
    int32_t w[CTL_WORDS];
    LS_TRY(read_ctl(m, w));
    if (w[CTL_STATUS]) return LS_ERR_DEVICE_STATUS;
    float ms = 0.f;
    LS_CK(cudaEventElapsedTime(&ms, m->ev0, m->ev1));
    m->stats.prefill_ms = ms;
    off = 0;
    for (int b = 0; b < n_seq; ++b) {
        m->b_n_prompt.push_back(prompt_lens[b]);
        m->b_last_tok.push_back(prompts[off + prompt_lens[b] - 1]);
        off += prompt_lens[b];
    }
    m->prefilled_layers = m->c.n_layers;
    return LS_OK;
}

int ls_decode_batch(ls_model* m, int32_t exit_layer, int32_t num_draft, int32_t max_new)
{
    if (!m || m->b_n_prompt.empty()) return LS_ERR_INVALID_ARG;
    const ls_config& c = m->c;
    const int B = (int)m->b_n_prompt.size(), L = c.n_layers;
    int E = exit_layer, d = num_draft;
    if (max_new < 1 || d < 0 || E < 0) return LS_ERR_INVALID_ARG;
    if (E == 0) {
        if (d != 0) return LS_ERR_INVALID_ARG;
        E = L;  // plain greedy, B sequences per pass
    } else {
        if (d < 1 || E > L - 1) return LS_ERR_INVALID_ARG;
        if (d > c.max_draft) return LS_ERR_CAPACITY;
    }
    if (B * (d + 1) > LS_MAX_ROWS) return LS_ERR_CAPACITY;
    const int pps = m->n_pages / B, cap = pps * c.page_size;
    for (int b = 0; b < B; ++b)
        if ((int64_t)m->b_n_prompt[b] + max_new + d + 1 > cap) return LS_ERR_CAPACITY;

    SeqView view(m, B, pps, cap, m->page_table);
    ls_model::G* g = nullptr;
    if (m->use_graphs) LS_TRY(get_graph(m, E, d, true, 0.f, &g));
    std::vector<int32_t> w((size_t)B * CTL_WORDS, 0);
    for (int b = 0; b < B; ++b) {
        int32_t* cb = w.data() + (size_t)b * CTL_WORDS;
        cb[CTL_CACHE_LEN] = m->b_n_prompt[b] - 1;
        cb[CTL_CUR_TOK] = m->b_last_tok[b];
        cb[CTL_MAX_NEW] = max_new;
        cb[CTL_EOS] = c.eos_id;
        cb[CTL_D_EFF] = kNoStop;
    }
    LS_CK(cudaMemcpyAsync(m->ctl, w.data(), sizeof(int32_t) * w.size(), cudaMemcpyHostToDevice, m->st));
    LS_CK(cudaStreamSynchronize(m->st));
    int64_t launched = 0;
    int syncs = 0, n_out_min = 0, steps_done = 0;
    LS_CK(cudaEventRecord(m->ev0, m->st));
    for (;;) {
        // as in the single-sequence loop, for the sequence that is furthest behind
        const int remaining = max_new - n_out_min;
        int steps = (remaining + d) / (d + 1);
        if (steps_done > 0 && n_out_min > 0) {
            const int64_t est = ((int64_t)remaining * steps_done + n_out_min - 1) / n_out_min;
            steps = (int)(est < 1 ? 1 : est);
        }
        for (int i = 0; i < steps; ++i) {
            if (g) {
                LS_CK(cudaGraphLaunch(g->exec, m->st));
                launched += g->nodes;
            } else {
                const int64_t before = m->launches;
                LS_TRY(enqueue_step(m, E, d, true, 0.f));
                launched += m->launches - before;
            }
        }
        LS_CK(cudaMemcpyAsync(w.data(), m->ctl, sizeof(int32_t) * w.size(), cudaMemcpyDeviceToHost, m->st));
        LS_CK(cudaStreamSynchronize(m->st));
        ++syncs;
        n_out_min = max_new;
        steps_done = 0;
        for (int b = 0; b < B; ++b) {
            const int32_t* cb = w.data() + (size_t)b * CTL_WORDS;
            if (cb[CTL_STATUS]) return LS_ERR_DEVICE_STATUS;
            if (cb[CTL_N_OUT] < n_out_min) n_out_min = cb[CTL_N_OUT];
            if (cb[CTL_N_STEPS] > steps_done) steps_done = cb[CTL_N_STEPS];
        }
        if (w[CTL_DONE]) break;
    }
    LS_CK(cudaEventRecord(m->ev1, m->st));
    LS_CK(cudaEventSynchronize(m->ev1));
    float ms = 0.f;
    LS_CK(cudaEventElapsedTime(&ms, m->ev0, m->ev1));

    m->b_out.assign(B, {});
    m->b_acc.assign(B, {});
    int64_t kb = 0, acc_sum = 0, n_gen = 0, wb_longest = 0;
    for (int b = 0; b < B; ++b) {
        const int32_t* cb = w.data() + (size_t)b * CTL_WORDS;
        m->b_out[b].resize(cb[CTL_N_OUT]);
        m->b_acc[b].resize(cb[CTL_N_STEPS]);
        LS_CK(cudaMemcpyAsync(m->b_out[b].data(), m->out_ids + (size_t)b * cap, sizeof(int32_t) * cb[CTL_N_OUT],
                              cudaMemcpyDeviceToHost, m->st));
        LS_CK(cudaMemcpyAsync(m->b_acc[b].data(), m->accepted + (size_t)b * cap, sizeof(int32_t) * cb[CTL_N_STEPS],
                              cudaMemcpyDeviceToHost, m->st));
    }
    LS_CK(cudaStreamSynchronize(m->st));
    // every weight byte is read once per pass for all sequences: the weights of the longest
    // sequence's steps; each sequence reads its own k, v rows
    for (int b = 0; b < B; ++b) {
        int64_t wb = 0, kbb = 0, ab = 0;
        schedule_bytes(c, E, d, true, m->b_n_prompt[b], m->b_acc[b].data(), nullptr, (int)m->b_acc[b].size(), &wb, &kbb, &ab);
        if (wb > wb_longest) wb_longest = wb;
        kb += kbb;
        acc_sum += ab;
        n_gen += (int64_t)m->b_out[b].size();
    }
    m->stats.decode_ms = ms;
    m->stats.weight_bytes = wb_longest;
    m->stats.kv_bytes = kb;
    m->stats.kernel_launches = launched;
    m->stats.n_generated = (int32_t)n_gen;
    m->stats.n_steps = steps_done;
    m->stats.n_accepted = (int32_t)acc_sum;
    m->stats.host_syncs = syncs;
    return LS_OK;
}

int ls_read_output_seq(ls_model* m, int32_t seq, int32_t* out_ids, int32_t* out_n, int32_t* accepted, int32_t* out_steps)
{
    if (!m || seq < 0 || seq >= (int)m->b_out.size()) return LS_ERR_INVALID_ARG;
    const std::vector<int32_t>&o = m->b_out[seq], &a = m->b_acc[seq];
    if (out_ids && !o.empty()) memcpy(out_ids, o.data(), sizeof(int32_t) * o.size());
    if (out_n) *out_n = (int32_t)o.size();
    if (accepted && !a.empty()) memcpy(accepted, a.data(), sizeof(int32_t) * a.size());
    if (out_steps) *out_steps = (int32_t)a.size();
    return LS_OK;
}

int ls_generate_batch(ls_model* m, int32_t n_seq, const int32_t* prompts, const int32_t* prompt_lens, int32_t exit_layer,
                      int32_t num_draft, int32_t max_new, int32_t* out_ids, int32_t* out_n, int32_t* accepted,
                      int32_t* out_steps)
{
    if (!m || !out_ids || !out_n || !accepted || !out_steps || max_new < 1) return LS_ERR_INVALID_ARG;
    LS_TRY(ls_prefill_batch(m, n_seq, prompts, prompt_lens));
    LS_TRY(ls_decode_batch(m, exit_layer, num_draft, max_new));
    for (int b = 0; b < n_seq; ++b)
        LS_TRY(ls_read_output_seq(m, b, out_ids + (size_t)b * max_new, out_n + b, accepted + (size_t)b * max_new, out_steps + b));
    return LS_OK;
}

int ls_debug_logits(ls_model* m, const int32_t* ids, int32_t n, int32_t exit_layer, float* exit_logits,
                    float* final_logits)
{
    if (!m) return LS_ERR_INVALID_ARG;
    LS_TRY(check_ids(m, ids, n));
    const int L = m->c.n_layers, V = m->c.vocab;
    if (exit_layer < 1 || exit_layer > L) return LS_ERR_INVALID_ARG;
    if (n > m->c.max_seq) return LS_ERR_CAPACITY;
    m->n_prompt = 0;
    LS_CK(cudaMemcpyAsync(m->ids, ids, sizeof(int32_t) * n, cudaMemcpyHostToDevice, m->st));
    LS_TRY(write_ctl(m, 0, 0, 0));
    for (int r0 = 0; r0 < n; r0 += kMaxRows) {
        int M = n - r0 < kMaxRows ? n - r0 : kMaxRows;
        LS_TRY(run_embed(m, m->ids + r0, M, m->x, 0));
        LS_TRY(run_layers(m, 0, exit_layer, M, m->x, r0, 0, m->h, m->fnorm,
                          exit_layer < L ? m->lw[exit_layer].attn_norm : nullptr));
        if (exit_logits) {
            LS_TRY(run_head(m, M, 0, m->verified, m->logits));
            LS_CK(cudaMemcpyAsync(exit_logits + (size_t)r0 * V, m->logits, sizeof(float) * (size_t)M * V,
                                  cudaMemcpyDeviceToHost, m->st));
            LS_CK(cudaStreamSynchronize(m->st));
        }
        if (exit_layer < L) LS_TRY(run_layers(m, exit_layer, L, M, m->x, r0, 0, m->hE, m->fnorm, nullptr));
        if (final_logits) {
            LS_TRY(run_head(m, M, 0, m->verified, m->logits));
            LS_CK(cudaMemcpyAsync(final_logits + (size_t)r0 * V, m->logits, sizeof(float) * (size_t)M * V,
                                  cudaMemcpyDeviceToHost, m->st));
            LS_CK(cudaStreamSynchronize(m->st));
        }
    }
    int32_t w[CTL_WORDS];
    LS_TRY(read_ctl(m, w));
    return w[CTL_STATUS] ? LS_ERR_DEVICE_STATUS : LS_OK;
}

int ls_debug_next_logits(ls_model* m, float* logits)
{
    if (!m || !logits || m->n_prompt < 1 || m->prefilled_layers < m->c.n_layers) return LS_ERR_INVALID_ARG;
    const ls_config& c = m->c;
    if (m->n_prompt + 1 > c.max_seq) return LS_ERR_CAPACITY;
    LS_TRY(write_ctl(m, m->n_prompt - 1, m->last_tok, 1));
    LS_TRY(run_embed(m, m->ctl + CTL_CUR_TOK, 1, m->x, 0));
    LS_TRY(run_layers(m, 0, c.n_layers, 1, m->x, 0, 0, m->h, m->fnorm, nullptr));
    LS_TRY(run_head(m, 1, 0, m->verified, m->logits));
    LS_CK(cudaMemcpyAsync(logits, m->logits, sizeof(float) * (size_t)c.vocab, cudaMemcpyDeviceToHost, m->st));
    int32_t w[CTL_WORDS];
    LS_TRY(read_ctl(m, w));
    return w[CTL_STATUS] ? LS_ERR_DEVICE_STATUS : LS_OK;
}

int ls_get_stats(const ls_model* m, ls_stats* out)
{
    if (!m || !out) return LS_ERR_INVALID_ARG;
    *out = m->stats;
    return LS_OK;
}

// ------------------------------------------------------------------ single operations
int ls_op_chain(int32_t on)
{
    g_op_chain = on != 0;
    return LS_OK;
}

int ls_op_embed(const void* emb, const int32_t* tok, int32_t M, int32_t D, int32_t V, float* x, void* stream)
{
    if (!aligned16(emb) || !tok || !aligned16(x) || M < 1 || M > LS_MAX_ROWS || D < 8 || D % 8 || V < 1)
        return LS_ERR_INVALID_ARG;
    LS_CK(launch(LaunchCtx{(cudaStream_t)stream, g_op_chain}, embed_kernel, dim3(M), dim3(256), 0, (const uint16_t*)emb, tok,
                 D, V, x, nullptr, nullptr, nullptr, nullptr, 0, 1));
    return LS_OK;
}

int ls_op_rmsnorm(const float* x, const void* gain, int32_t M, int32_t D, float eps, void* out, void* stream)
{
    if (!aligned16(x) || !aligned16(gain) || !aligned16(out) || M < 1 || M > LS_MAX_ROWS || D < 8 || D % 8)
        return LS_ERR_INVALID_ARG;
    LS_CK(launch(LaunchCtx{(cudaStream_t)stream, g_op_chain}, rmsnorm_kernel, dim3(M), dim3(256), 0, x,
                 (const uint16_t*)gain, D, eps, (uint16_t*)out, nullptr));
    return LS_OK;
}

static int lin_check(int path, const void* w, const void* h, int M, int N, int K)
{
    if (path != LS_LINEAR_FMA && path != LS_LINEAR_MMA) return LS_ERR_INVALID_ARG;
    if (!aligned16(w) || !aligned16(h) || M < 1 || M > LS_MAX_ROWS || N < 1 || K < 8 || K % 8) return LS_ERR_INVALID_ARG;
    return LS_OK;
}

int ls_op_linear(int32_t path, const void* w, const void* h, int32_t M, int32_t N, int32_t K, float* out,
                 int32_t residual, void* stream)
{
    LS_TRY(lin_check(path, w, h, M, N, K));
    if (!out) return LS_ERR_INVALID_ARG;
    LinArgs a = lin_args((const uint16_t*)w, (const uint16_t*)h, M, N, K);
    a.out = out;
    a.ldo = N;
    LS_CK(launch_linear(path, residual ? EPI_RESIDUAL : EPI_STORE, a, LaunchCtx{(cudaStream_t)stream, g_op_chain}));
    return LS_OK;
}

int ls_op_gate_up_swiglu(int32_t path, const void* wg, const void* wu, const void* h, int32_t M, int32_t F,
                         int32_t K, void* out, void* stream)
{
    LS_TRY(lin_check(path, wg, h, M, F, K));
    if (!aligned16(wu) || !out) return LS_ERR_INVALID_ARG;
    LinArgs a = lin_args((const uint16_t*)wg, (const uint16_t*)h, M, F, K);
    a.w1 = (const uint16_t*)wu;
    a.out_bf16 = (uint16_t*)out;
    LS_CK(launch_linear(path, EPI_SWIGLU, a, LaunchCtx{(cudaStream_t)stream, g_op_chain}));
    return LS_OK;
}

size_t ls_op_lm_head_scratch_bytes(int32_t V)
{
    if (V < 1) return 0;
    return sizeof(ValIdx) * (size_t)LS_MAX_ROWS * (size_t)((V + 15) / 16);
}

int ls_op_lm_head_argmax(int32_t path, const void* w, const void* h, int32_t M, int32_t V, int32_t K,
                         void* scratch, int32_t* tok, float* logits, void* stream)
{
    LS_TRY(lin_check(path, w, h, M, V, K));
    if (!scratch || ((uintptr_t)scratch & 7u) || !tok) return LS_ERR_INVALID_ARG;
    LinArgs a = lin_args((const uint16_t*)w, (const uint16_t*)h, M, V, K);
    a.cand = (ValIdx*)scratch;
    a.cand_stride = (V + 15) / 16;
    a.out = logits;
    a.ldo = V;
    const LaunchCtx lc = {(cudaStream_t)stream, g_op_chain};
    LS_CK(launch_linear(path, EPI_ARGMAX, a, lc));
    LS_CK(launch(lc, argmax_finish_kernel, dim3(M), dim3(256), 0, a.cand, n_candidates(path, V, K, M), a.cand_stride, tok,
                 nullptr, nullptr, 0.f, 0, 0ull));
    return LS_OK;
}

// ---- LM head + argmax without any allocation by anybody: the candidate buffer lives in
// the library image.  Every GPU that loads the library holds these bytes until exit.
static __device__ __align__(256) unsigned char g_lm_head_static_scratch[LS_OP_LM_HEAD_STATIC_BYTES];
static_assert(sizeof(ValIdx) * LS_MAX_ROWS * (LS_OP_LM_HEAD_STATIC_MAX_VOCAB / 16) == LS_OP_LM_HEAD_STATIC_BYTES,
              "one (value, index) candidate per 16 vocabulary rows and pass row");

// In host code the array's name is only a handle; its device address has to be asked for,
// once per device, with that device current.
static int static_scratch_address(void** out)
{
    constexpr int kMaxDevices = 64;
    static void* addr[kMaxDevices] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    LS_CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return LS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        LS_CK(cudaGetSymbolAddress(&p, g_lm_head_static_scratch));
        if (!p || ((uintptr_t)p & 255u)) return LS_ERR_UNSUPPORTED;
        addr[dev] = p;
    }
    *out = addr[dev];
    return LS_OK;
}

int ls_op_lm_head_argmax_static(int32_t path, const void* w, const void* h, int32_t M, int32_t V, int32_t K,
                                int32_t* tok, void* stream)
{
    LS_TRY(lin_check(path, w, h, M, V, K));
    if (!tok) return LS_ERR_INVALID_ARG;
    if (V > LS_OP_LM_HEAD_STATIC_MAX_VOCAB) return LS_ERR_CAPACITY;  // vocabulary beyond the built-in buffer
    void* scratch = nullptr;
    LS_TRY(static_scratch_address(&scratch));
    LinArgs a = lin_args((const uint16_t*)w, (const uint16_t*)h, M, V, K);
    a.cand = (ValIdx*)scratch;
    a.cand_stride = (V + 15) / 16;
    a.ldo = V;
    const LaunchCtx lc = {(cudaStream_t)stream, g_op_chain};
    LS_CK(launch_linear(path, EPI_ARGMAX, a, lc));
    LS_CK(launch(lc, argmax_finish_kernel, dim3(M), dim3(256), 0, a.cand, n_candidates(path, V, K, M), a.cand_stride, tok,
                 nullptr, nullptr, 0.f, 0, 0ull));
    return LS_OK;
}

static int kv_check(int M, int pos0, int Hq, int Hkv, int hd, int page_size, int max_seq)
{
    if (M < 1 || M > LS_MAX_ROWS || pos0 < 0 || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq / Hkv > 8) return LS_ERR_INVALID_ARG;
    if ((hd != 64 && hd != 128) || page_size < 16 || page_size > 1024 || log2_exact(page_size) < 0) return LS_ERR_INVALID_ARG;
    if (max_seq < 1 || max_seq > kAttnChunk * kAttnMaxChunks || (int64_t)pos0 + M > max_seq) return LS_ERR_CAPACITY;
    return LS_OK;
}

int ls_op_rope_append(const float* qkv, int32_t M, int32_t pos0, int32_t Hq, int32_t Hkv, int32_t hd, float theta,
                      int32_t page_size, const int32_t* page_table, int32_t max_seq, void* q_out, void* kp, void* vp,
                      void* stream)
{
    LS_TRY(kv_check(M, pos0, Hq, Hkv, hd, page_size, max_seq));
    if (!qkv || !page_table || !q_out || !aligned16(kp) || !aligned16(vp) || !(theta > 0.f)) return LS_ERR_INVALID_ARG;
    LS_CK(launch(LaunchCtx{(cudaStream_t)stream, g_op_chain}, rope_append_kernel, dim3(M, Hq + 2 * Hkv), dim3(hd / 2), 0, qkv,
                 Hq, Hkv, hd, nullptr, theta, log2_exact(page_size), page_table, max_seq, (uint16_t*)q_out, (uint16_t*)kp,
                 (uint16_t*)vp, nullptr, pos0));
    return LS_OK;
}

int ls_op_qkv_rope_append(int32_t path, const void* wq, const void* wk, const void* wv, const void* h, int32_t M,
                          int32_t K, int32_t pos0, int32_t Hq, int32_t Hkv, int32_t hd, float theta, int32_t page_size,
                          const int32_t* page_table, int32_t max_seq, void* q_out, void* kp, void* vp, void* stream)
{
    LS_TRY(kv_check(M, pos0, Hq, Hkv, hd, page_size, max_seq));
    LS_TRY(lin_check(path, wq, h, M, (Hq + 2 * Hkv) * hd, K));
    if (!aligned16(wk) || !aligned16(wv) || !page_table || !q_out || !aligned16(kp) || !aligned16(vp) || !(theta > 0.f))
        return LS_ERR_INVALID_ARG;
    LinArgs a = lin_args((const uint16_t*)wq, (const uint16_t*)h, M, (Hq + 2 * Hkv) * hd, K);
    a.w1 = (const uint16_t*)wk;
    a.w2 = (const uint16_t*)wv;
    a.n0 = Hq * hd;
    a.n1 = Hkv * hd;
    a.page_table = page_table;
    a.q_out = (uint16_t*)q_out;
    a.kpages = (uint16_t*)kp;
    a.vpages = (uint16_t*)vp;
    a.Hq = Hq;
    a.Hkv = Hkv;
    a.hd = hd;
    a.page_shift = log2_exact(page_size);
    a.max_seq = max_seq;
    a.pos_off = pos0;
    a.theta = theta;
    LS_CK(launch_linear(path, EPI_QKV, a, LaunchCtx{(cudaStream_t)stream, g_op_chain}));
    return LS_OK;
}

int ls_op_attention(const void* q, int32_t M, int32_t pos0, int32_t Hq, int32_t Hkv, int32_t hd, int32_t page_size,
                    const int32_t* page_table, int32_t max_seq, const void* kp, const void* vp, void* out, void* stream)
{
    LS_TRY(kv_check(M, pos0, Hq, Hkv, hd, page_size, max_seq));
    if (!aligned16(q) || !page_table || !aligned16(kp) || !aligned16(vp) || !out) return LS_ERR_INVALID_ARG;
    AttnPlan plan;
    LS_TRY(attn_plan(hd, Hq / Hkv, Hkv, max_seq, &plan));
    return attn_launch(plan, (const uint16_t*)q, (const uint16_t*)kp, (const uint16_t*)vp, page_table, nullptr, pos0, M,
                       Hq, Hkv, hd, log2_exact(page_size), max_seq, (uint16_t*)out, LaunchCtx{(cudaStream_t)stream, g_op_chain});
}

int ls_op_gemm(const void* a, const void* b, int32_t M, int32_t N, int32_t K, float* c, int32_t ldc, int32_t accumulate,
               int32_t* status_dev, void* stream)
{
    if (!aligned16(a) || !aligned16(b) || !c || M < 1 || N < 1 || K < 8 || K % 8 || ldc < N) return LS_ERR_INVALID_ARG;
    return gemm_launch((const uint16_t*)a, (const uint16_t*)b, M, N, K, c, ldc, accumulate, status_dev,
                       (cudaStream_t)stream);
}

int ls_op_prefill_attention(const void* q, int32_t R, int32_t pos0, int32_t Hq, int32_t Hkv, int32_t hd,
                            int32_t page_size, const int32_t* page_table, int32_t max_seq, const void* kp,
                            const void* vp, void* out, int32_t* status, void* stream)
{
    if (R < 1 || pos0 < 0 || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq / Hkv > 8 || (hd != 64 && hd != 128) ||
        page_size < 16 || page_size > 1024 || log2_exact(page_size) < 0)
        return LS_ERR_INVALID_ARG;
    if ((int64_t)pos0 + R > max_seq) return LS_ERR_CAPACITY;
    if (!aligned16(q) || !page_table || !aligned16(kp) || !aligned16(vp) || !out) return LS_ERR_INVALID_ARG;
    return prefill_attn_launch((const uint16_t*)q, (const uint16_t*)kp, (const uint16_t*)vp, page_table, pos0, R, Hq,
                               Hkv, hd, log2_exact(page_size), (max_seq + page_size - 1) / page_size, (uint16_t*)out, status,
                               (cudaStream_t)stream);
}

int ls_op_accept(const int32_t* draft, const int32_t* verified, int32_t d, int32_t* state, int32_t* out_ids,
                 int32_t* accepted, void* stream)
{
    if (!draft || !verified || !state || !out_ids || !accepted || d < 0 || d >= LS_MAX_ROWS) return LS_ERR_INVALID_ARG;
    LS_CK(launch(LaunchCtx{(cudaStream_t)stream, g_op_chain}, accept_kernel, dim3(1), dim3(32), 0, draft, verified, d, state,
                 out_ids, accepted, 0, nullptr));
    return LS_OK;
}


#ifdef LS_TRACE
// Timeline build (-DLS_TRACE, see ls_common.cuh): clear the records and switch recording on or off ...
int ls_trace_reset(int on)
{
    std::vector<TraceRec> z(kTraceSlots);
    for (auto& r : z) { r.key = 0; r.s0 = r.w0 = r.e0 = ~0ull; r.s1 = r.w1 = r.e1 = 0; r.n = 0; }
    LS_CK(cudaDeviceSynchronize());
    LS_CK(cudaMemcpyToSymbol(g_trace, z.data(), sizeof(TraceRec) * kTraceSlots));
    LS_CK(cudaMemcpyToSymbol(g_trace_on, &on, sizeof(int)));
    LS_CK(cudaDeviceSynchronize());
    return LS_OK;
}
// ... and copy the kTraceSlots records (8 x uint64 each) to the host
int ls_trace_read(void* out)
{
    LS_CK(cudaDeviceSynchronize());
    LS_CK(cudaMemcpyFromSymbol(out, g_trace, sizeof(TraceRec) * kTraceSlots));
    return LS_OK;
}
#endif

}  // extern "C"

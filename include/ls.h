/*
 * ls.h -- C ABI of the B200 (sm_100a) library for batch-1 self-speculative greedy
 * decoding on a Llama-style decoder (LayerSkip, arXiv 2404.16710, Sec. 4.3 and
 * Appendix A.4).
 *
 * Conventions for every entry point
 *   - "dev" pointers are CUDA device pointers on the current device, "host" pointers
 *     are ordinary host memory.  The library BORROWS every device pointer it is given
 *     (weights, workspace, operands): the caller allocates them, keeps them alive and
 *     frees them.  The library itself allocates no device memory.
 *   - bf16 matrices are row-major [out_features, in_features] and 16-byte aligned;
 *     in_features must be a multiple of 8.
 *   - Return value: LS_OK (0) or a negative ls_status.  No exception crosses the ABI,
 *     nothing aborts the process.  ls_strerror() names a status; after LS_ERR_CUDA,
 *     ls_last_cuda_error() returns the cudaError_t value seen.
 *   - A model handle is bound to one device and one stream; calls on one handle must
 *     not overlap.  Compute capability 10.x is required (LS_ERR_UNSUPPORTED otherwise);
 *     there is no CPU fallback.
 *   - Numerics: bf16 weights, bf16 KV cache, bf16 inputs of every linear layer, fp32
 *     residual stream and fp32 accumulation.  A row's result never depends on how many
 *     rows share the pass, so the verification pass (Sec. 4.3.2) reproduces
 *     single-token decoding bit for bit and ls_generate returns exactly the ids of
 *     ls_generate_full.
 */
#ifndef LS_B200_H
#define LS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ls_status {
    LS_OK = 0,
    LS_ERR_INVALID_ARG = -1,   /* null / misaligned pointer, value out of range            */
    LS_ERR_CAPACITY = -2,      /* KV capacity, workspace size or max_draft exceeded         */
    LS_ERR_CUDA = -3,          /* a CUDA runtime call failed; see ls_last_cuda_error()      */
    LS_ERR_DEVICE_STATUS = -4, /* a kernel's own bounds check refused an access             */
    LS_ERR_UNSUPPORTED = -5    /* not an sm_100 device, or a shape the kernels do not cover */
} ls_status;

#define LS_MAX_ROWS 16 /* rows (tokens) per pass: num_draft + 1 <= LS_MAX_ROWS */

/* Which kernel family runs every linear layer of a model.  The choice is per model,
 * never per call: results are bit-identical across M only within one family. */
enum { LS_LINEAR_AUTO = 0, LS_LINEAR_FMA = 1, LS_LINEAR_MMA = 2 };

/* Decoder shape (Sec. 4.1: L residual layers and the shared LM head g). */
typedef struct ls_config {
    int32_t n_layers;    /* L                                                            */
    int32_t d_model;     /* D, multiple of 8                                             */
    int32_t n_heads;     /* query heads Hq                                               */
    int32_t n_kv_heads;  /* KV heads Hkv, divides Hq, Hq/Hkv <= 8                        */
    int32_t head_dim;    /* 64 or 128                                                    */
    int32_t d_ffn;       /* F, multiple of 8                                             */
    int32_t vocab;       /* V                                                            */
    float rms_eps;
    float rope_theta;
    int32_t max_seq;     /* KV capacity in tokens (<= 16384): n_prompt+max_new+num_draft+1 */
    int32_t page_size;   /* tokens per KV page: power of two, 16..1024                   */
    int32_t max_draft;   /* largest num_draft this model will be asked for (<= 15)       */
    int32_t eos_id;      /* -1: never stop early                                         */
    int32_t linear_path; /* LS_LINEAR_*                                                  */
} ls_config;

/* Device pointers to the bf16 weights.  The per-layer members are HOST arrays of
 * n_layers device pointers.  Matrices [out, in]: wq [Hq*hd, D], wk/wv [Hkv*hd, D],
 * wo [D, Hq*hd], w_gate/w_up [F, D], w_down [D, F], tok_embed/lm_head [V, D];
 * norm gains are [D]. */
typedef struct ls_weights {
    const void *tok_embed, *final_norm, *lm_head;
    const void *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
    const void *const *ffn_norm, *const *w_gate, *const *w_up, *const *w_down;
} ls_weights;

typedef struct ls_model ls_model; /* opaque, owned by the library (host memory only) */

/* Counters of the most recent prefill / decode on a handle. */
typedef struct ls_stats {
    double prefill_ms;       /* device time of the prompt pass                              */
    double decode_ms;        /* device time of the decode loop (CUDA events on the stream)  */
    int64_t weight_bytes;    /* weight bytes the schedule had to read during decode         */
    int64_t kv_bytes;        /* KV-cache bytes the schedule had to read during decode       */
    int64_t kernel_launches; /* kernels launched by the decode loop                         */
    int32_t n_generated;
    int32_t n_steps;         /* speculative steps (== n_generated for plain greedy)         */
    int32_t n_accepted;      /* sum of accepted drafts over the steps                       */
    int32_t host_syncs;      /* host<->device synchronisations inside the decode loop       */
} ls_stats;

const char *ls_strerror(int status);
int ls_last_cuda_error(void);

/* Bytes of device workspace a model of this shape needs (KV pages, page table,
 * activations, exit-layer activation cache, control words).  0 if cfg is invalid. */
size_t ls_workspace_bytes(const ls_config *cfg);

/* Create a model over borrowed weights and workspace (256-byte aligned, at least
 * ls_workspace_bytes(cfg)).  cuda_stream is a cudaStream_t that can be captured into a
 * CUDA graph, i.e. not the legacy default stream; with NULL the model creates a (blocking)
 * stream of its own, which still runs after work already queued on the default stream.
 * The workspace is cleared; the page table starts as the identity. */
int ls_model_create(const ls_config *cfg, const ls_weights *w, void *workspace_dev,
                    size_t workspace_bytes, void *cuda_stream, ls_model **out);
int ls_model_destroy(ls_model *m);

/* Replace the logical->physical KV page table: host array of
 * ceil(max_seq/page_size) distinct physical page numbers in [0, n_pages). */
int ls_set_page_table(ls_model *m, const int32_t *table_host, int32_t n_pages);

/* Self-speculative greedy decoding (Sec. 4.3, Appendix A.4).
 * The prompt except its last token is run through all L layers; then every step
 *   drafts num_draft tokens with layers 0..E-1 and the shared LM head (Sec. 4.3.1),
 *   verifies them with layers E..L-1 in one pass of num_draft+1 rows that starts from
 *   the cached exit-layer activations and shares the KV cache (Sec. 4.3.2, 4.3.3),
 *   accepts the longest agreeing prefix plus the verified token after it and rolls the
 *   cache back to "every emitted token but the last" (Appendix A.4: match, crop).
 * prompt_ids_host [n_prompt]; exit_layer E in [1, L-1]; num_draft in [1, max_draft];
 * out_ids_host [max_new] receives *out_n <= max_new ids (fewer only after an EOS);
 * accepted_per_step_host [max_new] receives the accepted-draft count of each of the
 * *out_n_steps steps (the last one counted before truncation at max_new).
 * LS_ERR_CAPACITY if n_prompt + max_new + num_draft + 1 > max_seq. */
int ls_generate(ls_model *m, const int32_t *prompt_ids_host, int32_t n_prompt,
                int32_t exit_layer, int32_t num_draft, int32_t max_new,
                int32_t *out_ids_host, int32_t *out_n,
                int32_t *accepted_per_step_host, int32_t *out_n_steps);

/* Self-speculative decoding with an adaptive draft length.  The paper drafts a fixed number
 * of tokens per step and names dynamic, per-token conditions as future work (Sec. 9); this
 * entry point adds the simplest such condition, a confidence test on the exit logits, in the
 * way that keeps the method exact.  Within a step, draft pass j (j = 0 .. max_draft-1)
 * computes g(x_E) for its row; if the margin between the two largest exit logits,
 *     margin_j = logit_(1) - logit_(2)   (fp32, 0 on a tie),
 * is below min_margin, draft j is NOT kept and drafting stops: the step keeps k = j drafts
 * (possibly none).  Otherwise all max_draft drafts are kept and, as in ls_generate, one more
 * early pass prepares the last draft's row.  Verification then scores rows 0..k, accepts the
 * longest agreeing prefix of the k kept drafts and emits the verified token after it, so the
 * ids are still exactly those of ls_generate_full whatever min_margin is; only the number of
 * steps and the work per step change.  The exit-layer row of the discarded draft's input is
 * already computed, so stopping costs no extra pass.
 * min_margin > 0 (LS_ERR_INVALID_ARG otherwise; +inf keeps no draft at all, every step then
 * emits one token).  drafted_per_step_host [max_new] receives k of every step,
 * accepted_per_step_host the accepted count n <= k.  Other arguments and errors as
 * ls_generate with num_draft = max_draft. */
int ls_generate_adaptive(ls_model *m, const int32_t *prompt_ids_host, int32_t n_prompt,
                         int32_t exit_layer, int32_t max_draft, float min_margin, int32_t max_new,
                         int32_t *out_ids_host, int32_t *out_n, int32_t *accepted_per_step_host,
                         int32_t *drafted_per_step_host, int32_t *out_n_steps);

/* Autoregressive greedy decoding with all L layers: the baseline of Sec. 6.2 and,
 * by construction of the method, the exact result ls_generate must reproduce. */
int ls_generate_full(ls_model *m, const int32_t *prompt_ids_host, int32_t n_prompt,
                     int32_t max_new, int32_t *out_ids_host, int32_t *out_n);

/* Early-exit greedy decoding (Sec. 4.2): every token is argmax g(x_E). */
int ls_generate_early(ls_model *m, const int32_t *prompt_ids_host, int32_t n_prompt,
                      int32_t exit_layer, int32_t max_new, int32_t *out_ids_host, int32_t *out_n);

/* Several sequences through the loop together (the paper's Sec. 9 leaves batching to future
 * work; the loop itself is Sec. 4.3 / Appendix A.4, run per sequence).  Decoding one sequence is
 * bound by reading the weights; with B sequences every pass carries B rows (draft) or
 * B * (num_draft + 1) rows (verify), so each weight byte read from HBM serves all of them.
 * Each sequence drafts, verifies and accepts on its own: its own cache length, its own share
 * of the KV pages (n_pages / B pages, i.e. a capacity of (n_pages / B) * page_size positions),
 * its own accepted-per-step record; a sequence that reaches max_new (or EOS) stops emitting
 * while the others go on.  Every sequence's ids are bit-identical to what ls_generate_full
 * returns for its prompt alone on the same model.
 *   prompts_host      the prompts one after the other, prompt_lens_host[b] ids each
 *   exit_layer, num_draft   as in ls_generate; exit_layer == 0 and num_draft == 0: plain greedy
 *   out_ids_host      [n_seq][max_new], out_n[b] valid ids in row b
 *   accepted_per_step [n_seq][max_new], out_n_steps[b] valid entries in row b
 * Errors: LS_ERR_CAPACITY if n_seq * (num_draft + 1) > LS_MAX_ROWS, num_draft > max_draft or a
 * prompt + max_new + num_draft + 1 exceeds a sequence's share of the cache; LS_ERR_INVALID_ARG
 * for n_seq < 1, bad ids, exit_layer outside [1, L-1] with num_draft > 0.  The single-sequence
 * state left by ls_prefill is discarded (the sequences use its pages).
 * ls_prefill_batch / ls_decode_batch / ls_read_output_seq are the halves, as below. */
int ls_generate_batch(ls_model *m, int32_t n_seq, const int32_t *prompts_host,
                      const int32_t *prompt_lens_host, int32_t exit_layer, int32_t num_draft,
                      int32_t max_new, int32_t *out_ids_host, int32_t *out_n,
                      int32_t *accepted_per_step_host, int32_t *out_n_steps);
int ls_prefill_batch(ls_model *m, int32_t n_seq, const int32_t *prompts_host,
                     const int32_t *prompt_lens_host);
int ls_decode_batch(ls_model *m, int32_t exit_layer, int32_t num_draft, int32_t max_new);
int ls_read_output_seq(ls_model *m, int32_t seq, int32_t *out_ids_host, int32_t *out_n,
                       int32_t *accepted_per_step_host, int32_t *out_n_steps);

/* The two halves of a generate call, for callers that keep everything on the device
 * (and for timing the decode loop alone).  ls_prefill copies the prompt, runs
 * prompt[0..n-2] through the first `layers` layers (0 = all L; early-exit decoding
 * needs only E) and leaves the loop state at cache length n-1.  ls_decode runs the
 * loop from that state: exit_layer == 0 selects plain greedy with all layers,
 * num_draft == 0 with exit_layer > 0 selects early-exit greedy.  ls_decode may be
 * repeated after one ls_prefill: it restarts from the prefilled state every time.
 * Results stay on the device until ls_read_output. */
int ls_prefill(ls_model *m, const int32_t *prompt_ids_host, int32_t n_prompt, int32_t layers);
int ls_decode(ls_model *m, int32_t exit_layer, int32_t num_draft, int32_t max_new);
/* ls_decode with options.  LS_DECODE_NO_EXIT_CACHE is the paper's "without KVQ reuse" ablation
 * (Sec. 7, Table 7): the verify pass does not continue from the cached exit-layer
 * activations but runs all L layers on the num_draft+1 rows again.  Same ids, more bytes. */
#define LS_DECODE_NO_EXIT_CACHE 1
int ls_decode_flags(ls_model *m, int32_t exit_layer, int32_t num_draft, int32_t max_new, int32_t flags);
int ls_read_output(ls_model *m, int32_t *out_ids_host, int32_t *out_n,
                   int32_t *accepted_per_step_host, int32_t *out_n_steps);
/* The decode loop of ls_generate_adaptive from a prefilled state, and the kept-draft count of
 * every step of the last decode call (num_draft for the non-adaptive loops). */
int ls_decode_adaptive(ls_model *m, int32_t exit_layer, int32_t max_draft, float min_margin,
                       int32_t max_new);
int ls_read_drafted(ls_model *m, int32_t *drafted_per_step_host, int32_t *out_n_steps);

/* Teacher-forced logits for parity checks: feed ids_host[0..n-1] at positions 0..n-1
 * and return g(x_E) and g(x_L) for every position (host fp32 [n, V]; either may be
 * NULL).  g is the shared head of Sec. 2.1 / 4.2.  n <= max_seq. */
int ls_debug_logits(ls_model *m, const int32_t *ids_host, int32_t n, int32_t exit_layer,
                    float *exit_logits_host, float *final_logits_host);

/* Logits of the next token after ls_prefill (all layers): the last prompt token is run
 * through the model on top of the cache the prompt pass has left, g(x_L) goes to
 * logits_host (fp32 [V]).  For parity checks of the prompt pass itself: every layer's cached
 * k, v of every prompt position enters these logits.  The loop state is left as ls_prefill
 * left it (ls_decode may follow). */
int ls_debug_next_logits(ls_model *m, float *logits_host);

int ls_get_stats(const ls_model *m, ls_stats *out);

/* ------------------------------------------------------------------------------
 * Single operations of the path (each is one kernel family of the loop), exposed so
 * that each can be checked against its definition and profiled alone.  All pointers
 * are device pointers; M <= LS_MAX_ROWS rows; the call is enqueued on cuda_stream and
 * returns without synchronising.  linear_path is LS_LINEAR_FMA or LS_LINEAR_MMA.
 * ------------------------------------------------------------------------------ */

/* How the decode loop chains its kernels, for the single-operation calls below: with on != 0 every
 * later ls_op_* launch of this process carries the programmatic-dependent-launch attribute, so
 * consecutive operations on one stream overlap the way they do inside ls_generate (Sec. 4.3's
 * loop is one dependency chain): a kernel's CTAs may become resident and put their first weight
 * stages in flight while the operation before it on the stream is still running; every kernel
 * waits for that operation to finish before it touches anything but weights and the page table.
 * Results are unchanged.  Off by default (each operation then starts after the previous one has
 * drained, which is what a stand-alone timing of one kernel wants).  Process-wide, not per stream;
 * the prompt-pass kernels (ls_op_gemm, ls_op_prefill_attention) are not affected. */
int ls_op_chain(int32_t on);

/* x[m,:] = float(Emb[tok[m],:]) -- the embedding lookup x_0 of Sec. 4.1. */
int ls_op_embed(const void *emb_bf16_dev, const int32_t *tok_dev, int32_t M, int32_t D, int32_t V,
                float *x_dev, void *cuda_stream);

/* RMSNorm of each row: out[m,i] = bf16( x[m,i] / sqrt(mean_j x[m,j]^2 + eps) * g[i] ). */
int ls_op_rmsnorm(const float *x_dev, const void *gain_dev, int32_t M, int32_t D, float eps,
                  void *out_bf16_dev, void *cuda_stream);

/* out[m,n] = sum_k W[n,k] h[m,k]; W bf16 [N,K], h bf16 [M,K], out fp32 [M,N].
 * If residual != 0 the product is ADDED to out (the x <- x + f(x) update of Sec. 4.1). */
int ls_op_linear(int32_t linear_path, const void *w_dev, const void *h_bf16_dev, int32_t M,
                 int32_t N, int32_t K, float *out_dev, int32_t residual, void *cuda_stream);

/* SwiGLU feed-forward input: out[m,f] = bf16( silu(Wg h)[f] * (Wu h)[f] ). */
int ls_op_gate_up_swiglu(int32_t linear_path, const void *w_gate_dev, const void *w_up_dev,
                         const void *h_bf16_dev, int32_t M, int32_t F, int32_t K,
                         void *out_bf16_dev, void *cuda_stream);

/* Shared LM head fused with argmax (Sec. 2.1, Sec. 4.2): tok[m] = argmax_v (W h[m])_v,
 * the lowest index wins a tie.  scratch_dev: ls_op_lm_head_scratch_bytes(V) bytes.
 * logits_dev (fp32 [M,V]) may be NULL. */
size_t ls_op_lm_head_scratch_bytes(int32_t V);
int ls_op_lm_head_argmax(int32_t linear_path, const void *w_dev, const void *h_bf16_dev,
                         int32_t M, int32_t V, int32_t K, void *scratch_dev, int32_t *tok_dev,
                         float *logits_dev, void *cuda_stream);

/* The same operation for callers that cannot allocate device memory at all and so have
 * no scratch buffer to pass: code running between cudaStreamBeginCapture and EndCapture,
 * plug-ins and callbacks that are handed a stream but no allocator, and hosts whose
 * memory pool is sized up front and closed.  (The paper has no counterpart; this is a
 * convenience of this library.)  The per-CTA candidates go to a buffer that is part of
 * the library image, LS_OP_LM_HEAD_STATIC_BYTES bytes on every GPU that loads the
 * library, held until the process exits.  The call itself performs no cudaMalloc /
 * cudaFree and calls nothing that allocates.
 *   - V <= LS_OP_LM_HEAD_STATIC_MAX_VOCAB, otherwise LS_ERR_CAPACITY (nothing is launched).
 *   - The first call on each device looks up the buffer's device address (with that device
 *     current); make that first call outside any stream capture.  The first call of each kernel
 *     configuration (linear path, and the class of M, V and K) also sets a kernel attribute and
 *     loads the kernel: warm up with the same path and sizes as the calls that follow.
 *   - All calls share the one buffer and it keeps the previous call's contents.  Nothing
 *     in it has to start at zero: every candidate the finishing kernel reads is rewritten
 *     by the same call.  Two calls that may run on the GPU at the same time (different
 *     streams, no dependency) race on it -- order them.
 * Inputs and the tok_dev output are the caller's, as in ls_op_lm_head_argmax; there is no
 * logits output. */
#define LS_OP_LM_HEAD_STATIC_MAX_VOCAB 131072
#define LS_OP_LM_HEAD_STATIC_BYTES (8u * LS_MAX_ROWS * (LS_OP_LM_HEAD_STATIC_MAX_VOCAB / 16))
int ls_op_lm_head_argmax_static(int32_t linear_path, const void *w_dev, const void *h_bf16_dev,
                                int32_t M, int32_t V, int32_t K, int32_t *tok_dev,
                                void *cuda_stream);

/* Rotary embedding + KV append: rows m = 0..M-1 sit at positions pos0+m.  qkv fp32
 * [M, (Hq+2Hkv)*hd] (q heads, then k heads, then v heads).  Writes q_out bf16
 * [M, Hq*hd] and k, v (bf16) into the paged cache: k_pages / v_pages hold physical
 * pages of [Hkv][page_size][hd]; page_table_dev maps logical page -> physical page. */
int ls_op_rope_append(const float *qkv_dev, int32_t M, int32_t pos0, int32_t Hq, int32_t Hkv,
                      int32_t hd, float rope_theta, int32_t page_size, const int32_t *page_table_dev,
                      int32_t max_seq, void *q_out_bf16_dev, void *k_pages_dev, void *v_pages_dev,
                      void *cuda_stream);

/* The same, fused behind the q|k|v projection (what the decode loop runs): q, k, v =
 * W_q h, W_k h, W_v h for M rows of h (bf16 [M,K]; wq [Hq*hd,K], wk/wv [Hkv*hd,K]), then
 * rotary embedding and cache append as in ls_op_rope_append, with no fp32 round trip. */
int ls_op_qkv_rope_append(int32_t linear_path, const void *wq_dev, const void *wk_dev, const void *wv_dev,
                          const void *h_bf16_dev, int32_t M, int32_t K, int32_t pos0, int32_t Hq,
                          int32_t Hkv, int32_t hd, float rope_theta, int32_t page_size,
                          const int32_t *page_table_dev, int32_t max_seq, void *q_out_bf16_dev,
                          void *k_pages_dev, void *v_pages_dev, void *cuda_stream);

/* Causal attention of rows m at positions pos0+m over cache positions 0..pos0+m, with
 * grouped KV heads (query head i reads KV head i / (Hq/Hkv)): the one KV cache that the
 * draft and the verify stage share (Sec. 4.3.3).  q bf16 [M, Hq*hd]; out bf16 [M, Hq*hd].
 * One thread-block cluster per KV head; the cache is cut by absolute position into chunks of
 * 64 keys that are dealt out round-robin to the cluster's CTAs, each CTA keeps a running
 * (max, sum, weighted values) over its chunks and the CTAs' results are combined in CTA order
 * through distributed shared memory.  A row's result depends on its position only, never on M.
 * No scratch memory.  max_seq: capacity of the cache in tokens (<= 16384); it bounds the
 * positions (and, below 512, the cluster size: calls that are to agree bit for bit on caches
 * that small must pass the same value). */
int ls_op_attention(const void *q_bf16_dev, int32_t M, int32_t pos0, int32_t Hq, int32_t Hkv,
                    int32_t hd, int32_t page_size, const int32_t *page_table_dev, int32_t max_seq,
                    const void *k_pages_dev, const void *v_pages_dev, void *out_bf16_dev,
                    void *cuda_stream);

/* Kernels of the prompt pass (the rows that go through the model before the first draft,
 * Appendix A.4), which is a dense contraction over hundreds of rows.
 * ls_op_gemm: c[m, n] (+)= sum_k a[m, k] b[n, k] on the tcgen05 tensor cores (up to 128 rows
 * one CTA per 128 x 256 tile, beyond that persistent pairs of CTAs on 256 x 256 tiles with two
 * accumulators in tensor memory, so that a tile's epilogue overlaps the next tile's MMAs); a bf16 [M, K],
 * b bf16 [N, K], K a multiple of 8, both 16-byte aligned; c fp32 with leading dimension
 * ldc >= N; accumulate != 0 adds to c (the residual update of Sec. 4.1).  status_dev (device
 * int32, may be NULL) receives 3 if one of the kernel's bounded waits ran out.
 * ls_op_prefill_attention: causal attention of R rows at positions pos0 .. pos0+R-1 over the
 * paged cache (as ls_op_attention, any R, no scratch; the pools hold ceil(max_seq / page_size)
 * pages and every table entry is below that).  Head dim 128 and R >= 128: one CTA per (128 rows,
 * query head) on the tcgen05 tensor cores -- key blocks of 64, the scores, the softmax weights
 * and the running output in tensor memory, K and V by TMA from the pages, the softmax one row
 * per thread; status_dev (device int32, may be NULL) receives 3 if one of its bounded waits ran
 * out.  Otherwise a CTA walks the key chunks of its rows in order with a running max / sum per
 * row on mma.sync (status_dev is not written).  Keys at positions >= pos0 + R are never used,
 * whatever bits the pages hold there. */
int ls_op_gemm(const void *a_bf16_dev, const void *b_bf16_dev, int32_t M, int32_t N, int32_t K,
               float *c_dev, int32_t ldc, int32_t accumulate, int32_t *status_dev, void *cuda_stream);
int ls_op_prefill_attention(const void *q_bf16_dev, int32_t R, int32_t pos0, int32_t Hq, int32_t Hkv,
                            int32_t hd, int32_t page_size, const int32_t *page_table_dev,
                            int32_t max_seq, const void *k_pages_dev, const void *v_pages_dev,
                            void *out_bf16_dev, int32_t *status_dev, void *cuda_stream);

/* match + crop of Appendix A.4 on device arrays: n = number of leading i < d with
 * draft[i] == verified[i]; appends draft[0..n-1], verified[n] to out_ids (truncated at
 * max_new, and after the first eos_id if eos_id >= 0).
 * state_dev int32[8]: {cache_len, cur_token, n_out, n_steps, done, max_new, eos_id, status};
 * updated in place: cache_len += n+1, cur_token = verified[n], accepted[n_steps++] = n,
 * done = (n_out == max_new || EOS emitted). */
int ls_op_accept(const int32_t *draft_dev, const int32_t *verified_dev, int32_t d,
                 int32_t *state_dev, int32_t *out_ids_dev, int32_t *accepted_dev,
                 void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LS_B200_H */

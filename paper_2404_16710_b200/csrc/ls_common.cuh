// Shared device-side definitions of the decode kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ls {

// Control words of the decode loop, int32 in device memory.  Every kernel of the loop
// reads its positions from here, so one captured CUDA graph serves every step.
enum Ctl : int {
    CTL_CACHE_LEN = 0,  // tokens whose k, v are valid in the cache
    CTL_CUR_TOK = 1,    // input token of the next step (emitted, not yet cached)
    CTL_N_OUT = 2,      // ids emitted so far
    CTL_N_STEPS = 3,    // steps taken so far
    CTL_DONE = 4,       // loop finished: later kernels return at once
    CTL_MAX_NEW = 5,
    CTL_EOS = 6,
    CTL_STATUS = 7,     // non-zero: a kernel's bounds check refused an access
    CTL_D_EFF = 8,      // adaptive drafting: drafts this step keeps; kernels of draft pass j > this return at once
    CTL_SEQ_DONE = 9,   // several sequences per pass: this sequence has finished (CTL_DONE of block 0: all have)
    CTL_WORDS = 16
};
// Several sequences per pass (B of them): sequence b has its own block of control words at
// ctl + b * CTL_WORDS, its own pages (page table entries b * pt_stride ..) and its own output
// arrays.  Row r of a pass belongs to sequence r % B and is that sequence's row r / B, so the
// rows of one draft position are contiguous.  B = 1 is the single-sequence loop.
constexpr int kNoStop = 0x7fffffff;  // CTL_D_EFF while no draft pass has stopped the drafting

enum DevStatus : int { DEV_OK = 0, DEV_BAD_TOKEN = 1, DEV_POS_OVERFLOW = 2 };

constexpr int kMaxRows = 16;    // rows per pass
constexpr int kAttnChunk = 64;  // keys per attention chunk (absolute positions)

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float bf16f(uint16_t u) { return __uint_as_float(((uint32_t)u) << 16); }
__device__ __forceinline__ uint16_t f2bf(float f)
{
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    return (uint32_t)f2bf(lo) | ((uint32_t)f2bf(hi) << 16);
}

// Sums of squares for the RMSNorm that is carried across kernel boundaries are kept EXACT: every
// x^2 is rounded once to a multiple of 2^-32 and the multiples are added as 64-bit integers.
// Integer addition is associative, so the sum of a row does not depend on how the row's columns
// are dealt out to CTAs, warps and lanes -- kernels of any tiling leave the same bits, and a
// pass of several rows reproduces single-row decoding whatever configuration it runs in.
// Range: x^2 < 2^31 per element (saturating), row sums below 2^31 (rms up to ~700 at D = 4096).
__device__ __forceinline__ long long sq_fixed(float x) { return __float2ll_rn(x * x * 4294967296.0f); }
__device__ __forceinline__ float rms_rscale(long long ss, float inv_d, float eps)
{
    return 1.0f / sqrtf((float)ss * (1.0f / 4294967296.0f) * inv_d + eps);
}
// A row's sum is spread over kSsSlots accumulators (a CTA adds to slot blockIdx.x % kSsSlots)
// so that the hundreds of CTAs of a projection do not queue up on one address; a consumer adds
// the slots up -- in any order, the sum is exact.
constexpr int kSsSlots = 16;
__device__ __forceinline__ void ss_add(long long* row, long long v)
{
    atomicAdd(reinterpret_cast<unsigned long long*>(row + (blockIdx.x & (kSsSlots - 1))), (unsigned long long)v);
}
// Consumer side, called by the first 256 (or all, if fewer) threads of a CTA, whole warps: rs[m] =
// 1 / sqrt(mean x^2 + eps) of rows m < M (M * kSsSlots <= threads calling); with clear != nullptr
// CTA 0 zeroes the slots of the rows its successor's producer will add to.
__device__ __forceinline__ void rms_rscales(const long long* sums, long long* clear, int M, float inv_d, float eps,
                                            float* rs)
{
    const int i = threadIdx.x;
    long long v = 0;
    if (i < M * kSsSlots) {
        v = __ldcg(sums + i);
        if (clear && blockIdx.x == 0) clear[i] = 0;
    }
#pragma unroll
    for (int o = kSsSlots / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (i < M * kSsSlots && (i & (kSsSlots - 1)) == 0) rs[i / kSsSlots] = rms_rscale(v, inv_d, eps);
}

// 16-byte read of streamed-once data (weights): do not allocate in L1, so that the
// activations, which every CTA re-reads, stay there.
__device__ __forceinline__ uint4 ld_stream16(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// 16-byte read of small, heavily re-used data (activations): keep in L1.  A coherent load:
// the rows are written by the kernel before this one, which under programmatic dependent
// launch may still have been running when this kernel's CTAs started, so the read-only
// (non-coherent) path is not allowed for them.
__device__ __forceinline__ uint4 ld_reuse16(const void* p)
{
    uint4 v;
    asm volatile("ld.global.L1::evict_last.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead.
// .cg: L2 only (streamed weights); .ca: also L1 (activations, re-read by every CTA).
__device__ __forceinline__ void cp_async16_cg(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async16_ca(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds16(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// D (fp32, 16x8) += A (bf16, 16x16, row-major) * B (bf16, 16x8, "column-major": k contiguous per n)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// four 8x8 b16 matrices from shared memory, transposed on the way (lane L gives the row address
// L%8 of matrix L/8)
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// Programmatic dependent launch: a kernel launched with the attribute may start while its
// predecessor on the stream is still running.  pdl_wait() blocks until the predecessor
// grid has completed and its writes are visible; before it, a kernel may touch only
// memory that no kernel of the loop writes (weights, page table).  Without the launch
// attribute both are no-ops.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// every thread of every CTA of the cluster meets here; shared-memory writes made before it are
// visible to the cluster's other CTAs after it
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

#ifdef LS_TRACE
// ---- Timeline instrumentation, compiled in only with -DLS_TRACE (a separate library used by
// paper_2404_16710_b200/timeline.py; the product build carries none of it).  The linear and
// attention kernels stamp the global timer at CTA start, after the dependency wait and at CTA
// end; one CTA in eight folds its stamps into the record of its launch (first / last start,
// first / last wait release, first / last end).  A launch is identified by a pointer that is
// unique to it within one pass (its weight matrix, its layer's K pages) plus 1 for passes of
// more than one row; the record's slot is a hash of that key, which the host re-computes.
struct TraceRec { unsigned long long key, s0, s1, w0, w1, e0, e1, n; };
constexpr int kTraceSlots = 1 << 18;
__device__ TraceRec g_trace[kTraceSlots];
__device__ int g_trace_on;
__device__ __forceinline__ unsigned long long gtime()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__host__ __device__ __forceinline__ unsigned trace_hash(unsigned long long k)
{
    return (unsigned)((k * 0x9E3779B97F4A7C15ull) >> 40) & (unsigned)(kTraceSlots - 1);
}
__device__ __forceinline__ void tr_commit(const void* key, int sub, unsigned long long t0, unsigned long long t1)
{
    if (!*(volatile int*)&g_trace_on) return;
    const unsigned lin = blockIdx.x + blockIdx.y * gridDim.x, tot = gridDim.x * gridDim.y;
    if ((lin % 8) != 3 && lin != tot - 1 && lin != 0) return;
    const unsigned long long t2 = gtime();
    const unsigned long long k = (unsigned long long)key + (unsigned long long)sub;
    TraceRec* r = g_trace + trace_hash(k);
    atomicMax(&r->key, k);
    atomicMin(&r->s0, t0);
    atomicMax(&r->s1, t0);
    atomicMin(&r->w0, t1);
    atomicMax(&r->w1, t1);
    atomicMin(&r->e0, t2);
    atomicMax(&r->e1, t2);
    atomicAdd(&r->n, 1ull);
}
#define TR_T0 const unsigned long long tr0 = gtime();
#define TR_T1 const unsigned long long tr1 = gtime();
#define TR_END(key, sub) if (threadIdx.x == 0) tr_commit(key, sub, tr0, tr1);
#else
#define TR_T0
#define TR_T1
#define TR_END(key, sub)
#endif

struct LaunchCtx {
    cudaStream_t st;
    bool pdl;  // allow the kernel to start before the previous kernel on st has finished
};

template <typename... P, typename... A>
inline cudaError_t launch(const LaunchCtx& lc, void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, A... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = lc.st;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &at;
    cfg.numAttrs = lc.pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

struct ValIdx {
    float v;
    int i;
};
// total order: larger value first, then lower index (ties go to the lowest index)
__device__ __forceinline__ bool better(float v, int i, float bv, int bi)
{
    return v > bv || (v == bv && i < bi);
}
// best (v, idx) and second-largest value s of a growing set: one more element ...
__device__ __forceinline__ void top2_push(float x, int n, float& v, int& idx, float& s)
{
    if (better(x, n, v, idx)) {
        s = v;
        v = x;
        idx = n;
    } else {
        s = fmaxf(s, x);
    }
}
// ... or the union with a disjoint set whose best is (v2, i2) and whose second value is s2
__device__ __forceinline__ void top2_merge(float v2, int i2, float s2, float& v, int& idx, float& s)
{
    if (better(v2, i2, v, idx)) {
        s = fmaxf(v, s2);
        v = v2;
        idx = i2;
    } else {
        s = fmaxf(s, v2);
    }
}

// True when this launch has nothing to do: the loop is finished, or the launch belongs to
// draft pass `gate` (0: not a draft pass) and the step stopped drafting before it.
__device__ __forceinline__ bool pass_idle(const int32_t* ctl, int gate)
{
    return ctl && (ctl[CTL_DONE] || (gate > 0 && gate > ctl[CTL_D_EFF]));
}

}  // namespace ls

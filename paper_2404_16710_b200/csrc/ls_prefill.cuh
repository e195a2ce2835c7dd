// The prompt pass (everything before the decode loop starts): hundreds to thousands of
// rows at once, so its projections are real dense contractions and run on the 5th-gen
// tensor cores -- TMA tiles into 128B-swizzled shared memory, tcgen05.mma issued by one
// thread with the fp32 accumulator in tensor memory, tcgen05.ld for the epilogue.  Both
// ls_generate and ls_generate_full start from this same pass, so it needs no bit-for-bit
// relation to the small-M decode kernels; it only has to fill the KV cache the way the
// model defines it (LayerSkip Sec. 4.1 for the decoder; the appendix listing feeds the
// prompt through the model before the first draft).
#pragma once
#include <cuda.h>

#include "ls_kernels.cuh"

namespace ls {

// ------------------------------------------------------------------ small PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait: false if the phase did not complete within the poll budget (about a second).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
        if (it > 1024) __nanosleep(200);
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16 inputs, fp32 accumulate
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) and
// 128B-swizzled as TMA wrote them: 8-row groups 1024 bytes apart (stride byte offset),
// leading byte offset unused for swizzled K-major (1), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// ------------------------------------------------------------------ GEMM: C[M,N] (+)= A[M,K] B[N,K]^T
// Tile 128 x 256: with 128 x 128 tiles the kernel was bound by what the SMs can pull out of L2
// (32 KB of operands per 4 MMAs and SM; ~600 TFLOP/s whatever the grid), the wider tile moves
// 25 % fewer operand bytes per flop.
constexpr int kGemmBM = 128, kGemmBN = 256, kGemmBK = 64, kGemmStages = 4;
constexpr int kGemmStageBytes = (kGemmBM + kGemmBN) * kGemmBK * 2;                   // 48 KB
constexpr size_t kGemmSmemBytes = (size_t)kGemmStages * kGemmStageBytes + 1024 + 256;  // + alignment + barriers
constexpr int DEV_TIMEOUT = 3;

// Up to three B matrices with the same K in one launch (q|k|v, gate|up): their output columns
// follow one another in C.  A column tile belongs to one matrix (tiles do not straddle).
struct GemmSegs {
    int n[3];  // rows of B0, B1, B2 (0: unused)
};

// grid (column tiles of all matrices, ceil(M/128)), block 128.  Warp 0 allocates tensor memory
// and its lane 0 feeds the ring with TMA; lane 0 of warp 1 issues the MMAs; all four warps read
// their 32 accumulator lanes back and store (accumulate != 0: add to C, the residual update).
// Rows beyond M or N and columns beyond K come out of TMA as zeros.  Every wait is bounded; on
// a time-out the kernel records DEV_TIMEOUT in *status, still frees its tensor memory, returns.
__global__ void __launch_bounds__(128)
gemm_bf16_tn_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
                    const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
                    const GemmSegs segs, int M, int K, float* __restrict__ C, int ldc, int accumulate,
                    int32_t* status)
{
    extern __shared__ unsigned char gsm_raw[];
    const uint32_t base = (smem_u32(gsm_raw) + 1023u) & ~1023u;  // swizzled tiles want 1024-byte alignment
    const uint32_t bars = base + kGemmStages * kGemmStageBytes;  // full[S], empty[S], accum, tmem slot
    auto full = [&](int s) { return bars + 8u * s; };
    auto empty = [&](int s) { return bars + 8u * (kGemmStages + s); };
    const uint32_t accum = bars + 8u * (2 * kGemmStages);
    const uint32_t tslot = accum + 8u;
    __shared__ int failed;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.y * kGemmBM;
    // which matrix, which of its column tiles, where its columns start in C
    const CUtensorMap* map_b = &map_b0;
    int N = segs.n[0], n0 = blockIdx.x * kGemmBN, col0 = 0;
    {
        const int t0 = (segs.n[0] + kGemmBN - 1) / kGemmBN, t1 = (segs.n[1] + kGemmBN - 1) / kGemmBN;
        if ((int)blockIdx.x >= t0 + t1) {
            map_b = &map_b2;
            N = segs.n[2];
            n0 = ((int)blockIdx.x - t0 - t1) * kGemmBN;
            col0 = segs.n[0] + segs.n[1];
        } else if ((int)blockIdx.x >= t0) {
            map_b = &map_b1;
            N = segs.n[1];
            n0 = ((int)blockIdx.x - t0) * kGemmBN;
            col0 = segs.n[0];
        }
    }
    const int nkb = (K + kGemmBK - 1) / kGemmBK;
    if (tid == 0) {
        for (int s = 0; s < kGemmStages; ++s) {
            mbar_init(full(s), 1);
            mbar_init(empty(s), 1);
        }
        mbar_init(accum, 1);
        failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tslot), "r"(kGemmBN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    uint32_t tmem;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem) : "r"(tslot));

    if (warp == 0 && lane == 0) {  // TMA producer
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % kGemmStages;
            if (kb >= kGemmStages && !mbar_wait(empty(s), ((kb / kGemmStages) - 1) & 1)) {
                failed = 1;
                break;
            }
            mbar_expect_tx(full(s), kGemmStageBytes);
            const uint32_t sa = base + s * kGemmStageBytes, sb = sa + kGemmBM * kGemmBK * 2;
            tma_load_2d(sa, &map_a, kb * kGemmBK, m0, full(s));
            tma_load_2d(sb, map_b, kb * kGemmBK, n0, full(s));
        }
    } else if (warp == 1 && lane == 0) {  // MMA issuer
        // instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 128
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kGemmBN >> 3) << 17) |
                               ((uint32_t)(kGemmBM >> 4) << 24);
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % kGemmStages;
            if (!mbar_wait(full(s), (kb / kGemmStages) & 1)) {
                failed = 1;
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t sa = base + s * kGemmStageBytes, sb = sa + kGemmBM * kGemmBK * 2;
            const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sb);
#pragma unroll
            for (int k4 = 0; k4 < kGemmBK / 16; ++k4)  // 32 bytes (16 bf16) further along K per MMA
                tc_mma_bf16(tmem, da + 2 * k4, db + 2 * k4, idesc, (kb | k4) != 0);
            tc_commit(empty(s));  // arrives once these MMAs have finished reading the stage
        }
        tc_commit(accum);
    }
    __syncwarp();

    // epilogue: warp w owns accumulator lanes 32w..32w+31 = rows m0 + 32w + lane
    bool have = mbar_wait(accum, 0);
    if (!have) failed = 1;
    tc_fence_after();
    __syncthreads();
    if (!failed) {
        const int row = m0 + warp * 32 + lane;
#pragma unroll 1
        for (int c = 0; c < kGemmBN / 32; ++c) {
            uint32_t v[32];
            tc_ld32(tmem + ((uint32_t)(warp * 32) << 16) + c * 32, v);
            if (row < M) {
                float* dst = C + (size_t)row * ldc + col0 + n0 + c * 32;
                if (n0 + c * 32 + 32 <= N && (((uintptr_t)dst) & 15u) == 0) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float4 o = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                               __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                        if (accumulate) {
                            const float4 p = *reinterpret_cast<const float4*>(dst + j);
                            o.x += p.x;
                            o.y += p.y;
                            o.z += p.z;
                            o.w += p.w;
                        }
                        *reinterpret_cast<float4*>(dst + j) = o;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n0 + c * 32 + j < N) dst[j] = accumulate ? dst[j] + __uint_as_float(v[j]) : __uint_as_float(v[j]);
                }
            }
        }
    } else if (tid == 0 && status) {
        *status = DEV_TIMEOUT;
        __nanosleep(1000000);  // let copies that may still be in flight land before the CTA goes away
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kGemmBN) : "memory");
}

// ------------------------------------------------------------------ the same GEMM on CTA pairs
// Two CTAs of a cluster (2 x 1 x 1: neighbours along M) compute one 256 x 256 tile with
// tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of A and HALF of the weight tile
// (128 of the 256 rows of B), the leader CTA (cluster rank 0) issues the MMAs, which read both
// CTAs' shared memory and write each CTA's 128 x 256 accumulator into its own tensor memory.
// A weight byte is fetched from L2 once per 256 output rows instead of once per 128, so the
// operand traffic per flop is two thirds of the single-CTA kernel's.
//   - both CTAs' TMA loads signal the LEADER's full barrier (the .cta_group::2 form of the load;
//     the barrier address with the peer bit cleared), on which the leader expects both shares;
//   - tcgen05.commit multicasts to the barrier at the same offset in both CTAs (stage free,
//     accumulator ready);
//   - tensor memory is allocated and freed with the .cta_group::2 forms by warp 0 of both CTAs,
//     and the two CTAs meet at a cluster barrier after the barrier set-up and before freeing
//     (a CTA's shared memory must outlive the MMAs that read it).
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = (kGemmBM + kGemmBN / 2) * kGemmBK * 2;                    // 32 KB per CTA
constexpr size_t kPairSmemBytes = (size_t)kPairStages * kPairStageBytes + 1024 + 256;
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;  // shared::cluster address of the pair's even CTA

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t leader_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(leader_bar)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)  // arrives on `bar` in both CTAs of the pair
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3)
                 : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The kernel is persistent: grid = one CTA pair per two SMs, cluster (2, 1, 1), block 192.  Every
// pair walks a list of tiles (pair p takes tiles p, p + P, p + 2P, ...; rows fastest, so the
// pairs that run side by side share a weight tile in L2) and the roles live in warps of their
// own: warps 0-3 read accumulators back and store, lane 0 of warp 4 feeds the ring with TMA,
// lane 0 of warp 5 (leader CTA) issues the MMAs.  Tensor memory holds TWO accumulators (2 x 256 of its 512 columns): while the epilogue
// warps drain tile i, the MMAs of tile i + 1 already fill the other one, and the operand ring
// never drains between tiles.  Two more barrier pairs carry that: accf[b] "accumulator b is
// complete" (tcgen05.commit, multicast to both CTAs) and acce[b] "accumulator b has been read"
// (in the leader CTA; the eight epilogue warps of the pair arrive on it, the peer's through the
// cluster's shared-memory window).  Every wait is bounded as in the one-tile kernels.
// q|k|v epilogue of the prompt pass: instead of fp32 C, the rotary embedding is applied to the
// accumulator and q goes out as bf16 [M, Hq hd], k and v into the paged cache at positions
// pos0 + row (B0 = W_q, B1 = W_k, B2 = W_v).  A 256-column tile holds whole heads (hd 64 or 128), and
// the two halves of a rotary pair (j, j + hd/2) are two 32-column reads of the thread's accumulator
// row.  The angles come from a table of (cos, sin)(pos * theta^(-2j/hd)) filled once per model by
// rope_table_kernel with the arithmetic of the decode kernels.  q_out == nullptr: not this mode.
struct RopeEpi {
    const float2* table;  // [max_seq][hd/2]
    const int32_t* page_table;
    uint16_t *q_out, *kpages, *vpages;
    int Hq, Hkv, hd, page_shift, max_seq, pos0;
};

// grid (positions), block hd/2
__global__ void rope_table_kernel(const float* __restrict__ inv_freq, int half, float2* __restrict__ table)
{
    const int pos = blockIdx.x, j = threadIdx.x;
    if (j < half) {
        float sn, cs;
        sincosf((float)pos * inv_freq[j], &sn, &cs);
        table[(size_t)pos * half + j] = make_float2(cs, sn);
    }
}

constexpr int kPersistThreads = 192;
constexpr int kPersistTmemCols = 2 * kGemmBN;

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

__global__ void __launch_bounds__(kPersistThreads)
gemm_bf16_tn_pair_persistent_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b0,
                                    const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_b2,
                                    const GemmSegs segs, int M, int K, float* __restrict__ C, int ldc, int accumulate,
                                    int32_t* status, uint16_t* __restrict__ swiglu_out, const RopeEpi rope)
{
    extern __shared__ unsigned char gsm_raw[];
    const uint32_t base = (smem_u32(gsm_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + kPairStages * kPairStageBytes;  // full[S], empty[S], accf[2], acce[2], tmem slot
    auto full = [&](int s) { return bars + 8u * s; };
    auto empty = [&](int s) { return bars + 8u * (kPairStages + s); };
    auto accf = [&](int b) { return bars + 8u * (2 * kPairStages + b); };
    auto acce = [&](int b) { return bars + 8u * (2 * kPairStages + 2 + b); };
    const uint32_t tslot = bars + 8u * (2 * kPairStages + 4);
    __shared__ int failed;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const bool swiglu = swiglu_out != nullptr;
    const int t0 = (segs.n[0] + kGemmBN - 1) / kGemmBN, t1 = (segs.n[1] + kGemmBN - 1) / kGemmBN,
              t2 = (segs.n[2] + kGemmBN - 1) / kGemmBN;
    const int col_tiles = swiglu ? (segs.n[0] + kGemmBN / 2 - 1) / (kGemmBN / 2) : t0 + t1 + t2;
    const int row_pairs = ((M + kGemmBM - 1) / kGemmBM + 1) / 2;
    const int n_tiles = col_tiles * row_pairs;
    const int n_pairs = (int)gridDim.x / 2, pair = (int)blockIdx.x / 2;
    const int nkb = (K + kGemmBK - 1) / kGemmBK;

    // column tile ny -> weight matrix, its row count, first row of the tile in it, first output column
    struct Cols {
        const CUtensorMap* map;
        int N, n0, col0;
    };
    auto cols_of = [&](int ny) {
        Cols c;
        if (swiglu) {
            // the pair's weight tile is 128 gate rows (staged by the leader) beside the 128 up rows of
            // the same features (staged by its peer): the accumulator holds gate | up of 128 features
            c.map = rank ? &map_b1 : &map_b0;
            c.N = segs.n[0];
            c.n0 = ny * (kGemmBN / 2);
            c.col0 = 0;
        } else if (ny >= t0 + t1) {
            c.map = &map_b2;
            c.N = segs.n[2];
            c.n0 = (ny - t0 - t1) * kGemmBN;
            c.col0 = segs.n[0] + segs.n[1];
        } else if (ny >= t0) {
            c.map = &map_b1;
            c.N = segs.n[1];
            c.n0 = (ny - t0) * kGemmBN;
            c.col0 = segs.n[0];
        } else {
            c.map = &map_b0;
            c.N = segs.n[0];
            c.n0 = ny * kGemmBN;
            c.col0 = 0;
        }
        return c;
    };

    if (tid == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(full(s), 1);
            mbar_init(empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf(b), 1);
            mbar_init(acce(b), 8);  // four epilogue warps in each CTA of the pair
        }
        failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tslot), "r"(kPersistTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything signals them
    tc_fence_after();
    uint32_t tmem;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem) : "r"(tslot));

    if (warp == 4) {
        if (lane == 0) {  // TMA producer of this CTA's share
            int it = 0;
            bool ok = true;
            for (int t = pair; t < n_tiles && ok; t += n_pairs) {
                const Cols c = cols_of(t / row_pairs);
                const int m0 = ((t % row_pairs) * 2 + (int)rank) * kGemmBM;
                const int b_row = swiglu ? c.n0 : c.n0 + (int)rank * (kGemmBN / 2);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (it >= kPairStages && !mbar_wait(empty(s), ((it / kPairStages) - 1) & 1)) {
                        failed = 1;
                        ok = false;
                        break;
                    }
                    if (rank == 0) mbar_expect_tx(full(s), 2 * kPairStageBytes);
                    const uint32_t sa = base + s * kPairStageBytes, sb = sa + kGemmBM * kGemmBK * 2;
                    const uint32_t lead = full(s) & kPeerBitMask;
                    tma_load_2d_pair(sa, &map_a, kb * kGemmBK, m0, lead);
                    tma_load_2d_pair(sb, c.map, kb * kGemmBK, b_row, lead);
                }
            }
        }
    } else if (warp == 5) {
        if (rank == 0 && lane == 0) {  // MMA issuer: the leader CTA only
            // instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 256 (128 per CTA)
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kGemmBN >> 3) << 17) |
                                   ((uint32_t)((2 * kGemmBM) >> 4) << 24);
            int it = 0, i = 0;
            bool ok = true;
            for (int t = pair; t < n_tiles && ok; t += n_pairs, ++i) {
                const int b = i & 1;
                // accumulator b free: its previous tile (i - 2) has been read by all eight warps
                if (i >= 2 && !mbar_wait(acce(b), ((i >> 1) - 1) & 1)) {
                    failed = 1;
                    break;
                }
                tc_fence_after();
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kPairStages;
                    if (!mbar_wait(full(s), (it / kPairStages) & 1)) {
                        failed = 1;
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t sa = base + s * kPairStageBytes, sb = sa + kGemmBM * kGemmBK * 2;
                    const uint64_t da = umma_desc_sw128(sa), db = umma_desc_sw128(sb);
#pragma unroll
                    for (int k4 = 0; k4 < kGemmBK / 16; ++k4)
                        tc_mma_bf16_pair(tmem + (uint32_t)(b * kGemmBN), da + 2 * k4, db + 2 * k4, idesc, (kb | k4) != 0);
                    tc_commit_pair(empty(s));
                }
                if (ok) tc_commit_pair(accf(b));
            }
        }
    } else {
        // epilogue: warp w of each CTA owns its accumulator lanes 32w..32w+31 = rows m0 + 32w + lane
        const uint32_t acce_leader[2] = {cluster_map(acce(0), 0), cluster_map(acce(1), 0)};
        int i = 0;
        for (int t = pair; t < n_tiles; t += n_pairs, ++i) {
            const int b = i & 1;
            const Cols c = cols_of(t / row_pairs);
            const int N = c.N, n0 = c.n0, col0 = c.col0;
            const int row = ((t % row_pairs) * 2 + (int)rank) * kGemmBM + warp * 32 + lane;
            if (!mbar_wait(accf(b), (i >> 1) & 1)) {
                failed = 1;
                break;
            }
            tc_fence_after();
            const uint32_t tacc = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * kGemmBN);
            if (swiglu) {
#pragma unroll 1
                for (int cc = 0; cc < kGemmBN / 64; ++cc) {  // 32 features at a time: gate columns cc*32.., up columns 128 + cc*32..
                    uint32_t gt[32], up[32];
                    tc_ld32(tacc + cc * 32, gt);
                    tc_ld32(tacc + kGemmBN / 2 + cc * 32, up);
                    if (row < M) {
                        uint16_t* dst = swiglu_out + (size_t)row * N + n0 + cc * 32;
                        if (n0 + cc * 32 + 32 <= N && (((uintptr_t)dst) & 15u) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float g0 = __uint_as_float(gt[j + 2 * e]), g1 = __uint_as_float(gt[j + 2 * e + 1]);
                                    pk[e] = pack_bf16(g0 / (1.0f + expf(-g0)) * __uint_as_float(up[j + 2 * e]),
                                                      g1 / (1.0f + expf(-g1)) * __uint_as_float(up[j + 2 * e + 1]));
                                }
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + cc * 32 + j < N) {
                                    const float g0 = __uint_as_float(gt[j]);
                                    dst[j] = f2bf(g0 / (1.0f + expf(-g0)) * __uint_as_float(up[j]));
                                }
                        }
                    }
                }
            } else if (rope.q_out) {
                // whole heads of q, k or v (the tile's matrix says which): rotate pairs, convert, store
                const int hd = rope.hd, half = hd >> 1, pos = rope.pos0 + row;
                const int seg = col0 == 0 ? 0 : (col0 == segs.n[0] ? 1 : 2);  // 0: q, 1: k, 2: v
                const bool row_ok = row < M && pos >= 0 && pos < rope.max_seq;
                if (row < M && !row_ok && status) *status = DEV_POS_OVERFLOW;
#pragma unroll 1
                for (int hh = 0; hh < kGemmBN / hd; ++hh) {
                    const int head = (n0 + hh * hd) / hd;  // head within its matrix
                    uint16_t* dst = nullptr;
                    if (row_ok && n0 + hh * hd < N) {
                        if (seg == 0) dst = rope.q_out + ((size_t)row * rope.Hq + head) * hd;
                        else
                            dst = (seg == 1 ? rope.kpages : rope.vpages) +
                                  kv_row_offset(rope.page_table, pos, rope.page_shift, rope.Hkv, head, hd);
                    }
#pragma unroll 1
                    for (int cc = 0; cc < half / 32; ++cc) {
                        uint32_t lo[32], hi[32];
                        tc_ld32(tacc + hh * hd + cc * 32, lo);
                        tc_ld32(tacc + hh * hd + half + cc * 32, hi);
                        if (dst) {
                            const float2* tb = rope.table + (size_t)pos * half + cc * 32;
#pragma unroll
                            for (int j = 0; j < 32; j += 8) {
                                uint32_t pl[4], ph[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    float a0 = __uint_as_float(lo[j + 2 * e]), a1 = __uint_as_float(lo[j + 2 * e + 1]);
                                    float b0 = __uint_as_float(hi[j + 2 * e]), b1 = __uint_as_float(hi[j + 2 * e + 1]);
                                    if (seg != 2) {
                                        const float4 t = *reinterpret_cast<const float4*>(tb + j + 2 * e);  // cos, sin, cos, sin
                                        const float r0 = a0 * t.x - b0 * t.y, s0 = a0 * t.y + b0 * t.x;
                                        const float r1 = a1 * t.z - b1 * t.w, s1 = a1 * t.w + b1 * t.z;
                                        a0 = r0;
                                        b0 = s0;
                                        a1 = r1;
                                        b1 = s1;
                                    }
                                    pl[e] = pack_bf16(a0, a1);
                                    ph[e] = pack_bf16(b0, b1);
                                }
                                *reinterpret_cast<uint4*>(dst + cc * 32 + j) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
                                *reinterpret_cast<uint4*>(dst + half + cc * 32 + j) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
                            }
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int cc = 0; cc < kGemmBN / 32; ++cc) {
                    uint32_t v[32];
                    tc_ld32(tacc + cc * 32, v);
                    if (row < M) {
                        float* dst = C + (size_t)row * ldc + col0 + n0 + cc * 32;
                        if (n0 + cc * 32 + 32 <= N && (((uintptr_t)dst) & 15u) == 0) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4) {
                                float4 o = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                       __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                                if (accumulate) {
                                    const float4 q = *reinterpret_cast<const float4*>(dst + j);
                                    o.x += q.x;
                                    o.y += q.y;
                                    o.z += q.z;
                                    o.w += q.w;
                                }
                                *reinterpret_cast<float4*>(dst + j) = o;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + cc * 32 + j < N)
                                    dst[j] = accumulate ? dst[j] + __uint_as_float(v[j]) : __uint_as_float(v[j]);
                        }
                    }
                }
            }
            // this warp has read its lanes of accumulator b: tell the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acce_leader[b]);
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (failed && tid == 0 && status) {
        *status = DEV_TIMEOUT;
        __nanosleep(1000000);  // let copies that may still be in flight land before the CTA goes away
    }
    cluster_sync_all();  // both CTAs are done with tensor memory, and the MMAs with both shared memories
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kPersistTmemCols) : "memory");
}

// ------------------------------------------------------------------ elementwise helpers of the prompt pass
// a[m, f] = bf16(silu(gu[m, f]) * gu[m, F + f]); grid (rows), block 256; four features per
// thread and step when F allows 16-byte accesses
__global__ void __launch_bounds__(256)
swiglu_rows_kernel(const float* __restrict__ gu, int F, uint16_t* __restrict__ a)
{
    const float* g = gu + (size_t)blockIdx.x * 2 * F;
    uint16_t* o = a + (size_t)blockIdx.x * F;
    if ((F & 3) == 0) {
        for (int f = threadIdx.x * 4; f < F; f += 256 * 4) {
            const float4 x = *reinterpret_cast<const float4*>(g + f);
            const float4 u = *reinterpret_cast<const float4*>(g + F + f);
            uint2 r;
            r.x = pack_bf16(x.x / (1.0f + expf(-x.x)) * u.x, x.y / (1.0f + expf(-x.y)) * u.y);
            r.y = pack_bf16(x.z / (1.0f + expf(-x.z)) * u.z, x.w / (1.0f + expf(-x.w)) * u.w);
            *reinterpret_cast<uint2*>(o + f) = r;
        }
    } else {
        for (int f = threadIdx.x; f < F; f += 256) {
            const float x = g[f];
            o[f] = f2bf(x / (1.0f + expf(-x)) * g[F + f]);
        }
    }
}

// Rotary embedding and KV append for a block of prompt rows: qkv fp32 [R][(Hq + 2 Hkv) hd] ->
// q bf16 [R][Hq hd], k and v into the paged cache at positions pos0 + row.  grid (rows),
// block 256: a thread keeps one rotary pair index j and walks the heads, so the sine and
// cosine of its angle are computed once per row.  Same arithmetic as rope_append_kernel.
__global__ void __launch_bounds__(256)
rope_append_rows_kernel(const float* __restrict__ qkv, int Hq, int Hkv, int hd, const float* __restrict__ inv_freq,
                        int page_shift, const int32_t* __restrict__ page_table, int max_seq, int pos0,
                        uint16_t* __restrict__ q_out, uint16_t* __restrict__ kpages, uint16_t* __restrict__ vpages,
                        int32_t* status)
{
    const int m = blockIdx.x, half = hd >> 1;
    const int pos = pos0 + m;
    if (pos < 0 || pos >= max_seq) {
        if (status && threadIdx.x == 0) *status = DEV_POS_OVERFLOW;
        return;
    }
    const int j = threadIdx.x % half, h0 = threadIdx.x / half, hstep = 256 / half;
    float sn, cs;
    sincosf((float)pos * inv_freq[j], &sn, &cs);
    const int H = Hq + 2 * Hkv;
    const float* src = qkv + (size_t)m * H * hd;
    for (int h = h0; h < H; h += hstep) {
        float a = src[(size_t)h * hd + j], b = src[(size_t)h * hd + j + half];
        if (h < Hq + Hkv) {
            const float ra = a * cs - b * sn, rb = a * sn + b * cs;
            a = ra;
            b = rb;
        }
        uint16_t* dst;
        if (h < Hq) dst = q_out + ((size_t)m * Hq + h) * hd;
        else if (h < Hq + Hkv) dst = kpages + kv_row_offset(page_table, pos, page_shift, Hkv, h - Hq, hd);
        else dst = vpages + kv_row_offset(page_table, pos, page_shift, Hkv, h - Hq - Hkv, hd);
        dst[j] = f2bf(a);
        dst[j + half] = f2bf(b);
    }
}

// ------------------------------------------------------------------ causal attention of the prompt pass
// (The two kernels below serve head dim 64, blocks of fewer than 128 rows and group sizes beyond 4;
// head dim 128 with at least 128 rows runs on tcgen05, see ls_prefill_attn.cuh.)
// grid (ceil(R/16), Hkv), block 256.  CTA = 16 consecutive rows (positions pos0 + 16 b ..),
// KV head kh, its G query heads; it walks the key chunks 0 .. last visible in order with a
// running (max, sum, o) per query in shared memory -- no partials, no merge.
// shared memory: Ks | Vs | Qs f32 [Q][HD] | S f32 [Q][64] | O f32 [Q][HD] | mx, l, alpha f32 [Q] each
template <int HD>
__host__ __device__ constexpr size_t prefill_attn_smem_bytes(int Q)
{
    return (size_t)kAttnChunk * (HD * 2 + 64) + (size_t)kAttnChunk * (HD * 2 + 32) +
           sizeof(float) * (2 * (size_t)Q * HD + (size_t)Q * kAttnChunk + 3 * (size_t)Q);
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads)
prefill_attn_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ kpages,
                    const uint16_t* __restrict__ vpages, const int32_t* __restrict__ page_table, int pos0, int R,
                    int Hq, int Hkv, int page_shift, uint16_t* __restrict__ out)
{
    constexpr int C = kAttnChunk, T = kAttnThreads;
    constexpr int KROW = HD * 2 + 64, VROW = HD * 2 + 32, HALF = HD / 2, NKS = T / HALF;
    const int tid = threadIdx.x, kh = blockIdx.y;
    const int r0 = blockIdx.x * 16;
    const int M = min(16, R - r0);
    const int G = Hq / Hkv, Q = G * M;
    const int first_pos = pos0 + r0, last_pos = first_pos + M - 1;

    extern __shared__ __align__(16) unsigned char smem[];
    unsigned char* Ks = smem;
    unsigned char* Vs = Ks + C * KROW;
    float* Qs = reinterpret_cast<float*>(Vs + C * VROW);
    float* S = Qs + (size_t)Q * HD;
    float* O = S + (size_t)Q * C;
    float* mx = O + (size_t)Q * HD;
    float* ls = mx + Q;
    float* al = ls + Q;

    for (int idx = tid; idx < Q * HALF; idx += T) {
        const int qi = idx / HALF, dp = idx % HALF;
        const int m = qi / G, g = qi % G;
        const uint32_t u =
            *reinterpret_cast<const uint32_t*>(q + ((size_t)(r0 + m) * Hq + (size_t)kh * G + g) * HD + 2 * dp);
        Qs[2 * idx] = bf16lo(u);
        Qs[2 * idx + 1] = bf16hi(u);
        O[2 * idx] = 0.f;
        O[2 * idx + 1] = 0.f;
    }
    for (int qi = tid; qi < Q; qi += T) {
        mx[qi] = -INFINITY;
        ls[qi] = 0.f;
    }

    const int nch = last_pos / C + 1;
    const float scale = rsqrtf((float)HD);
    for (int ch = 0; ch < nch; ++ch) {
        const int key0 = ch * C;
        __syncthreads();  // previous chunk's K, V, S are no longer read
        {
            constexpr int SEGS = HD * 2 / 16;
            const uint32_t ks0 = smem_u32(Ks), vs0 = smem_u32(Vs);
            for (int idx = tid; idx < C * SEGS; idx += T) {
                const int r = idx / SEGS, sg = idx % SEGS;
                const int p = key0 + r;
                const bool ok = p <= last_pos;
                const size_t off = kv_row_offset(page_table, ok ? p : key0, page_shift, Hkv, kh, HD) + (size_t)sg * 8;
                cp_async16_cg(ks0 + r * KROW + sg * 16, kpages + off, ok ? 16 : 0);
                cp_async16_cg(vs0 + r * VROW + sg * 16, vpages + off, ok ? 16 : 0);
            }
            cp_async_commit();
            cp_async_wait<0>();
        }
        __syncthreads();
        {
            const int key = tid >> 2, qd = tid & 3;
            const unsigned char* krow = Ks + key * KROW;
            int q0 = 0;
            for (; q0 + 4 <= Q; q0 += 4) attn_qk<HD, 4>(krow, Qs, q0, qd, S, key, qd == 0);
            for (; q0 < Q; ++q0) attn_qk<HD, 1>(krow, Qs, q0, qd, S, key, qd == 0);
        }
        __syncthreads();
        {
            const int warp = tid >> 5, lane = tid & 31;
            for (int qi = warp; qi < Q; qi += T / 32) {
                const int pos = first_pos + qi / G;
                float s0 = S[(size_t)qi * C + lane] * scale;
                float s1 = S[(size_t)qi * C + lane + 32] * scale;
                if (key0 + lane > pos) s0 = -INFINITY;
                if (key0 + lane + 32 > pos) s1 = -INFINITY;
                float cm = fmaxf(s0, s1);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
                const float mo = mx[qi], mn = fmaxf(mo, cm);
                const float p0 = (s0 == -INFINITY) ? 0.f : expf(s0 - mn);
                const float p1 = (s1 == -INFINITY) ? 0.f : expf(s1 - mn);
                float l = p0 + p1;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                S[(size_t)qi * C + lane] = p0;
                S[(size_t)qi * C + lane + 32] = p1;
                if (lane == 0) {
                    const float a = (mn == -INFINITY) ? 1.f : ((mo == -INFINITY) ? 0.f : expf(mo - mn));
                    al[qi] = a;
                    ls[qi] = ls[qi] * a + l;
                    mx[qi] = mn;
                }
            }
        }
        __syncthreads();
        {
            const int ks = tid % NKS, dp = tid / NKS;
            int q0 = 0;
            for (; q0 + 4 <= Q; q0 += 4) {
                float o[4][2];
                attn_pv<HD, 4, NKS>(Vs, S, q0, dp, ks, o);
                if (ks == 0) {
#pragma unroll
                    for (int qq = 0; qq < 4; ++qq) {
                        float* dst = O + (size_t)(q0 + qq) * HD + 2 * dp;
                        const float a = al[q0 + qq];
                        dst[0] = dst[0] * a + o[qq][0];
                        dst[1] = dst[1] * a + o[qq][1];
                    }
                }
            }
            for (; q0 < Q; ++q0) {
                float o[1][2];
                attn_pv<HD, 1, NKS>(Vs, S, q0, dp, ks, o);
                if (ks == 0) {
                    float* dst = O + (size_t)q0 * HD + 2 * dp;
                    const float a = al[q0];
                    dst[0] = dst[0] * a + o[0][0];
                    dst[1] = dst[1] * a + o[0][1];
                }
            }
        }
    }
    __syncthreads();
    for (int idx = tid; idx < Q * HALF; idx += T) {
        const int qi = idx / HALF, dp = idx % HALF;
        const int m = qi / G, g = qi % G;
        const float l = ls[qi];
        *reinterpret_cast<uint32_t*>(out + ((size_t)(r0 + m) * Hq + (size_t)kh * G + g) * HD + 2 * dp) =
            pack_bf16(O[2 * idx] / l, O[2 * idx + 1] / l);
    }
}

// Causal attention of a block of prompt rows on the tensor cores (G = Hq / Hkv in {1, 2, 4}),
// in the flash-attention arrangement: a CTA of four warps takes 64 queries of one KV head
// (64 / G rows x G query heads), each warp 16 rows of one query head.  A warp keeps its
// queries as mma.sync A fragments, walks the 64-key chunks that all warps stage together
// (cp.async, two buffers: the next chunk travels while this one is used), and needs nobody
// else: s = q.k lands in accumulator registers, the running max / sum of its rows live in
// registers (quad shuffles), p is rounded to bf16 and is, in the accumulator layout, already
// the A fragment of p.v; the running output (16 x HD fp32) is rescaled per chunk.
// Scores are scaled by log2(e)/sqrt(hd) so that the exponentials are exp2.
// shared memory: 2 x (K [64][HD*2+16] | V [64][HD*2+16])
constexpr int kFaThreads = 128;
template <int HD>
__host__ __device__ constexpr size_t prefill_attn_fa_smem_bytes()
{
    return 2 * 2 * (size_t)kAttnChunk * (HD * 2 + 16);
}

template <int HD>
__global__ void __launch_bounds__(kFaThreads)
prefill_attn_fa_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ kpages,
                       const uint16_t* __restrict__ vpages, const int32_t* __restrict__ page_table, int pos0, int R,
                       int Hq, int Hkv, int page_shift, uint16_t* __restrict__ out)
{
    constexpr int C = kAttnChunk, T = kFaThreads;
    constexpr int ROW = HD * 2 + 16;   // bytes per staged row: conflict-free for both operand reads
    constexpr int SEGS = HD * 2 / 16;  // 16-byte pieces per row
    constexpr int KS = HD / 16;        // k-steps of q.k
    constexpr int NT = HD / 8;         // n8 tiles of the output
    constexpr int BUF = 2 * C * ROW;   // one buffer: K then V
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int kh = blockIdx.y, G = Hq / Hkv;
    const int rows_per_cta = 64 / G;
    const int r0 = blockIdx.x * rows_per_cta;
    const int M = min(rows_per_cta, R - r0);
    const int gq = warp % G, rt = warp / G;  // the warp's query head within the group, its tile of 16 rows
    const int head = kh * G + gq;
    const bool active = rt * 16 < M;
    const int last_pos = pos0 + r0 + M - 1;
    const int nch = last_pos / C + 1;
    const int warp_nch = active ? (pos0 + r0 + min(rt * 16 + 15, M - 1)) / C + 1 : 0;
    const int rowA = rt * 16 + g, rowB = rowA + 8;  // within the CTA's rows
    const int posA = pos0 + r0 + rowA, posB = posA + 8;

    // the warp's queries as A fragments (zeros for rows that do not exist)
    uint32_t qf[KS][4];
    {
        const uint16_t* qa = q + ((size_t)(r0 + min(rowA, M - 1)) * Hq + head) * HD;
        const uint16_t* qb = q + ((size_t)(r0 + min(rowB, M - 1)) * Hq + head) * HD;
        const bool va = active && rowA < M, vb = active && rowB < M;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
            qf[kk][0] = va ? *reinterpret_cast<const uint32_t*>(qa + kk * 16 + 2 * t) : 0u;
            qf[kk][1] = vb ? *reinterpret_cast<const uint32_t*>(qb + kk * 16 + 2 * t) : 0u;
            qf[kk][2] = va ? *reinterpret_cast<const uint32_t*>(qa + kk * 16 + 2 * t + 8) : 0u;
            qf[kk][3] = vb ? *reinterpret_cast<const uint32_t*>(qb + kk * 16 + 2 * t + 8) : 0u;
        }
    }
    const uint32_t sm0 = smem_u32(smem);
    const bool one_page = page_shift >= 6;
    auto stage = [&](int ch, int b) {  // rows of chunk ch -> buffer b (zeros beyond the last visible key)
        const int key0 = ch * C;
        const size_t base = one_page ? kv_row_offset(page_table, key0, page_shift, Hkv, kh, HD) : 0;
        const uint32_t kb = sm0 + b * BUF, vb = kb + C * ROW;
#pragma unroll
        for (int it = 0; it < C * SEGS / T; ++it) {
            const int idx = tid + it * T;
            const int r = idx / SEGS, sg = idx % SEGS;
            const int p = key0 + r;
            const bool ok = p <= last_pos;
            const size_t off = (one_page ? base + (size_t)r * HD
                                         : kv_row_offset(page_table, ok ? p : key0, page_shift, Hkv, kh, HD)) +
                               (size_t)sg * 8;
            cp_async16_cg(kb + r * ROW + sg * 16, kpages + off, ok ? 16 : 0);
            cp_async16_cg(vb + r * ROW + sg * 16, vpages + off, ok ? 16 : 0);
        }
    };

    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[nt][i] = 0.f;
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;  // running max; this thread's share of the sums
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
    const int mi = lane >> 3, mr = lane & 7;  // ldmatrix: lane -> row mr of matrix mi

    stage(0, 0);
    cp_async_commit();
    for (int ch = 0; ch < nch; ++ch) {
        if (ch + 1 < nch) stage(ch + 1, (ch + 1) & 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        if (ch < warp_nch) {
            const unsigned char* Kb = smem + (ch & 1) * BUF;
            const uint32_t vb = sm0 + (ch & 1) * BUF + C * ROW;
            float s[C / 8][4];
#pragma unroll
            for (int nt = 0; nt < C / 8; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) s[nt][i] = 0.f;
#pragma unroll
            for (int kk = 0; kk < KS; ++kk)
#pragma unroll
                for (int nt = 0; nt < C / 8; ++nt) {
                    const unsigned char* kr = Kb + (nt * 8 + g) * ROW + (kk * 16 + 2 * t) * 2;
                    mma_bf16_16816(s[nt], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3],
                                   *reinterpret_cast<const uint32_t*>(kr), *reinterpret_cast<const uint32_t*>(kr + 16));
                }
            // scale, causal mask, running max
            float cA = -INFINITY, cB = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < C / 8; ++nt) {
                const int key = ch * C + nt * 8 + 2 * t;
                s[nt][0] = key <= posA ? s[nt][0] * sc : -INFINITY;
                s[nt][1] = key + 1 <= posA ? s[nt][1] * sc : -INFINITY;
                s[nt][2] = key <= posB ? s[nt][2] * sc : -INFINITY;
                s[nt][3] = key + 1 <= posB ? s[nt][3] * sc : -INFINITY;
                cA = fmaxf(cA, fmaxf(s[nt][0], s[nt][1]));
                cB = fmaxf(cB, fmaxf(s[nt][2], s[nt][3]));
            }
            cA = fmaxf(cA, __shfl_xor_sync(0xffffffffu, cA, 1));
            cA = fmaxf(cA, __shfl_xor_sync(0xffffffffu, cA, 2));
            cB = fmaxf(cB, __shfl_xor_sync(0xffffffffu, cB, 1));
            cB = fmaxf(cB, __shfl_xor_sync(0xffffffffu, cB, 2));
            const float nA = fmaxf(mA, cA), nB = fmaxf(mB, cB);
            // (a row sees key 0 in its first chunk, so nA, nB are finite from then on)
            const float fA = nA == -INFINITY ? 0.f : nA, fB = nB == -INFINITY ? 0.f : nB;
            const float aA = exp2f(mA - fA), aB = exp2f(mB - fB);
            mA = nA;
            mB = nB;
            float pA = 0.f, pB = 0.f;
#pragma unroll
            for (int nt = 0; nt < C / 8; ++nt) {
                s[nt][0] = exp2f(s[nt][0] - fA);
                s[nt][1] = exp2f(s[nt][1] - fA);
                s[nt][2] = exp2f(s[nt][2] - fB);
                s[nt][3] = exp2f(s[nt][3] - fB);
                pA += s[nt][0] + s[nt][1];
                pB += s[nt][2] + s[nt][3];
            }
            lA = lA * aA + pA;
            lB = lB * aB + pB;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                o[nt][0] *= aA;
                o[nt][1] *= aA;
                o[nt][2] *= aB;
                o[nt][3] *= aB;
            }
            // o += p.v: p (bf16) in the accumulator layout is the A fragment
#pragma unroll
            for (int k2 = 0; k2 < C / 16; ++k2) {
                const uint32_t a0 = pack_bf16(s[2 * k2][0], s[2 * k2][1]), a1 = pack_bf16(s[2 * k2][2], s[2 * k2][3]);
                const uint32_t a2 = pack_bf16(s[2 * k2 + 1][0], s[2 * k2 + 1][1]);
                const uint32_t a3 = pack_bf16(s[2 * k2 + 1][2], s[2 * k2 + 1][3]);
                const uint32_t vrow = vb + (uint32_t)((k2 * 16 + (mi & 1) * 8 + mr) * ROW + (mi >> 1) * 16);
#pragma unroll
                for (int np = 0; np < NT / 2; ++np) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(vrow + np * 32, b0, b1, b2, b3);
                    mma_bf16_16816(o[2 * np], a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(o[2 * np + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        }
        __syncthreads();  // the buffer may be overwritten by the copy issued in the next round
    }
    if (!active) return;
    lA += __shfl_xor_sync(0xffffffffu, lA, 1);
    lA += __shfl_xor_sync(0xffffffffu, lA, 2);
    lB += __shfl_xor_sync(0xffffffffu, lB, 1);
    lB += __shfl_xor_sync(0xffffffffu, lB, 2);
    if (rowA < M) {
        uint16_t* dst = out + ((size_t)(r0 + rowA) * Hq + head) * HD + 2 * t;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) *reinterpret_cast<uint32_t*>(dst + nt * 8) = pack_bf16(o[nt][0] / lA, o[nt][1] / lA);
    }
    if (rowB < M) {
        uint16_t* dst = out + ((size_t)(r0 + rowB) * Hq + head) * HD + 2 * t;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) *reinterpret_cast<uint32_t*>(dst + nt * 8) = pack_bf16(o[nt][2] / lB, o[nt][3] / lB);
    }
}

}  // namespace ls

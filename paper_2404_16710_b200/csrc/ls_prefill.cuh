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

// The same walk on the tensor cores (used when a KV head's 16 rows x G query heads fit in four
// query tiles, G <= 4): q.k and p.v as mma.sync.m16n8k16 exactly as in the decode attention
// kernel (queries are the 16-row operand, V comes transposed out of ldmatrix), softmax pieces
// per chunk in fp32, the running output of every query tile stays in registers and is rescaled
// by exp(old max - new max) before each chunk's contribution is added.
// shared memory: Ks [64][HD*2+64] | Vs [64][HD*2+16] | Qb bf16 [Qpad][HD*2+64] | S f32 [Qpad][72]
//                | Pb bf16 [Qpad][72] | mx, l, alpha f32 [Qpad] each
template <int HD>
__host__ __device__ constexpr size_t prefill_attn_mma_smem_bytes(int Q)
{
    const size_t qpad = ((size_t)Q + 15) / 16 * 16;
    return (size_t)kAttnChunk * (HD * 2 + 64) + (size_t)kAttnChunk * (HD * 2 + 16) + qpad * (HD * 2 + 64) +
           qpad * kAttnSP * 4 + qpad * kAttnSP * 2 + 3 * qpad * sizeof(float);
}

template <int HD>
__global__ void __launch_bounds__(kAttnThreads)
prefill_attn_mma_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ kpages,
                        const uint16_t* __restrict__ vpages, const int32_t* __restrict__ page_table, int pos0, int R,
                        int Hq, int Hkv, int page_shift, uint16_t* __restrict__ out)
{
    constexpr int C = kAttnChunk, T = kAttnThreads;
    constexpr int KROW = HD * 2 + 64, VROW = HD * 2 + 16, SP = kAttnSP, PBROW = kAttnSP * 2;
    constexpr int SEGS = HD * 2 / 16;
    constexpr int NTW = HD / 64;  // n8 tiles of output dims per warp
    constexpr int MAXQT = 4;      // query tiles held in registers
    const int tid = threadIdx.x, kh = blockIdx.y;
    const int warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    const int r0 = blockIdx.x * 16;
    const int M = min(16, R - r0);
    const int G = Hq / Hkv, Q = G * M, Qpad = (Q + 15) & ~15;
    const int first_pos = pos0 + r0, last_pos = first_pos + M - 1;

    extern __shared__ __align__(16) unsigned char smem[];
    unsigned char* Ks = smem;
    unsigned char* Vs = Ks + C * KROW;
    unsigned char* Qb = Vs + C * VROW;
    float* S = reinterpret_cast<float*>(Qb + (size_t)Qpad * KROW);
    unsigned char* Pb = reinterpret_cast<unsigned char*>(S + (size_t)Qpad * SP);
    float* mx = reinterpret_cast<float*>(Pb + (size_t)Qpad * PBROW);
    float* ls = mx + Qpad;
    float* al = ls + Qpad;

    for (int idx = tid; idx < Qpad * SEGS; idx += T) {
        const int qi = idx / SEGS, sg = idx % SEGS;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (qi < Q) {
            const int m = qi / G, g = qi % G;
            v = *reinterpret_cast<const uint4*>(q + ((size_t)(r0 + m) * Hq + (size_t)kh * G + g) * HD + sg * 8);
        }
        *reinterpret_cast<uint4*>(Qb + qi * KROW + sg * 16) = v;
    }
    for (int qi = tid; qi < Qpad; qi += T) {
        mx[qi] = -INFINITY;
        ls[qi] = 0.f;
        al[qi] = 1.f;
    }
    float o[MAXQT][NTW][4];
#pragma unroll
    for (int qt = 0; qt < MAXQT; ++qt)
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[qt][nt][i] = 0.f;

    const int d0 = NTW * 8 * warp;
    const uint32_t ks0 = smem_u32(Ks), vs0 = smem_u32(Vs);
    const int mi = lane >> 3, mr = lane & 7;
    const uint32_t vlane = vs0 + (uint32_t)(((mi & 1) * 8 + mr) * VROW + (d0 + ((NTW == 2) ? (mi >> 1) * 8 : 0)) * 2);
    const float scale = rsqrtf((float)HD);
    const int nch = last_pos / C + 1;
    for (int ch = 0; ch < nch; ++ch) {
        const int key0 = ch * C;
        __syncthreads();  // the previous chunk's K, V, S, Pb are no longer read
        {
            const bool one_page = page_shift >= 6;
            const size_t base = one_page ? kv_row_offset(page_table, key0, page_shift, Hkv, kh, HD) : 0;
#pragma unroll
            for (int it = 0; it < C * SEGS / T; ++it) {
                const int idx = tid + it * T;
                const int r = idx / SEGS, sg = idx % SEGS;
                const int p = key0 + r;
                const bool ok = p <= last_pos;
                const size_t off = (one_page ? base + (size_t)r * HD
                                             : kv_row_offset(page_table, ok ? p : key0, page_shift, Hkv, kh, HD)) +
                                   (size_t)sg * 8;
                cp_async16_cg(ks0 + r * KROW + sg * 16, kpages + off, ok ? 16 : 0);
                cp_async16_cg(vs0 + r * VROW + sg * 16, vpages + off, ok ? 16 : 0);
            }
            cp_async_commit();
            cp_async_wait<0>();
        }
        __syncthreads();
        // s = q.k: warp w owns keys 8w..8w+7
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
            float* sp = S + (size_t)(qt + g8) * SP + 8 * warp + 2 * t4;
            *reinterpret_cast<float2*>(sp) = make_float2(c[0], c[1]);
            *reinterpret_cast<float2*>(sp + 8 * SP) = make_float2(c[2], c[3]);
        }
        __syncthreads();
        // per query: mask, running max and sum, p -> bf16
        for (int qi = warp; qi < Qpad; qi += T / 32) {
            uint16_t* pb = reinterpret_cast<uint16_t*>(Pb + (size_t)qi * PBROW);
            if (qi >= Q) {
                pb[lane] = 0;
                pb[lane + 32] = 0;
                continue;
            }
            const int pos = first_pos + qi / G;
            float s0 = S[(size_t)qi * SP + lane] * scale;
            float s1 = S[(size_t)qi * SP + lane + 32] * scale;
            if (key0 + lane > pos) s0 = -INFINITY;
            if (key0 + lane + 32 > pos) s1 = -INFINITY;
            float cm = fmaxf(s0, s1);
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, sh));
            const float mo = mx[qi], mn = fmaxf(mo, cm);
            const float p0 = (s0 == -INFINITY) ? 0.f : expf(s0 - mn);
            const float p1 = (s1 == -INFINITY) ? 0.f : expf(s1 - mn);
            float l = p0 + p1;
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) l += __shfl_xor_sync(0xffffffffu, l, sh);
            pb[lane] = f2bf(p0);
            pb[lane + 32] = f2bf(p1);
            if (lane == 0) {
                const float a = (mn == -INFINITY) ? 1.f : ((mo == -INFINITY) ? 0.f : expf(mo - mn));
                al[qi] = a;
                ls[qi] = ls[qi] * a + l;
                mx[qi] = mn;
            }
        }
        __syncthreads();
        // o = o * alpha + p.v: warp w owns output dims d0 .. d0 + 8 NTW - 1
#pragma unroll
        for (int qt = 0; qt < MAXQT; ++qt) {
            if (qt * 16 < Qpad) {
                float c[NTW][4];
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) c[nt][i] = 0.f;
                const unsigned char* pa = Pb + (size_t)(qt * 16 + g8) * PBROW + 4 * t4;
#pragma unroll
                for (int kk = 0; kk < C / 16; ++kk) {
                    const uint32_t a0 = *reinterpret_cast<const uint32_t*>(pa + 32 * kk);
                    const uint32_t a1 = *reinterpret_cast<const uint32_t*>(pa + 8 * PBROW + 32 * kk);
                    const uint32_t a2 = *reinterpret_cast<const uint32_t*>(pa + 32 * kk + 16);
                    const uint32_t a3 = *reinterpret_cast<const uint32_t*>(pa + 8 * PBROW + 32 * kk + 16);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(vlane + (uint32_t)(16 * kk * VROW), b0, b1, b2, b3);
                    mma_bf16_16816(c[0], a0, a1, a2, a3, b0, b1);
                    if (NTW == 2) mma_bf16_16816(c[NTW - 1], a0, a1, a2, a3, b2, b3);
                }
                const float alo = al[qt * 16 + g8], ahi = al[qt * 16 + g8 + 8];
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt) {
                    o[qt][nt][0] = o[qt][nt][0] * alo + c[nt][0];
                    o[qt][nt][1] = o[qt][nt][1] * alo + c[nt][1];
                    o[qt][nt][2] = o[qt][nt][2] * ahi + c[nt][2];
                    o[qt][nt][3] = o[qt][nt][3] * ahi + c[nt][3];
                }
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int qt = 0; qt < MAXQT; ++qt)
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {
            const int qi = qt * 16 + g8 + 8 * hrow;
            if (qi < Q) {
                const int m = qi / G, g = qi % G;
                const float l = ls[qi];
                uint16_t* dst = out + ((size_t)(r0 + m) * Hq + (size_t)kh * G + g) * HD + d0 + 2 * t4;
#pragma unroll
                for (int nt = 0; nt < NTW; ++nt)
                    *reinterpret_cast<uint32_t*>(dst + 8 * nt) =
                        pack_bf16(o[qt][nt][2 * hrow] / l, o[qt][nt][2 * hrow + 1] / l);
            }
        }
}

}  // namespace ls

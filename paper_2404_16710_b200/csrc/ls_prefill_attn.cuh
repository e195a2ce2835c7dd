// Causal attention of the prompt pass on the 5th-gen tensor cores (head dim 128).
//
// One CTA per (tile of 128 prompt rows, query head) walks the key blocks of 64 cache positions
// that its rows can see, as TWO independent online-softmax streams: stream A takes the even
// blocks, stream B the odd ones, each with two score buffers, its own running (max, sum) per row
// and its own output accumulator; the two are merged at the end like the spans of a split cache.
// Per block j of stream g = j mod 2 (buffer b = (j / 2) mod 2):
//   S_j = Q K_j^T      tcgen05.mma, 128 x 64 x 128, fp32 into S_{g,b} (tensor memory)
//   P_j = exp2(S_j c - m)   four warps, one query row per thread: the row of S_{g,b} by tcgen05.ld,
//                      running maximum m and sum l in registers, P_j rounded to bf16 and written
//                      back by tcgen05.st over the first 32 columns of S_{g,b} (two keys per word)
//   O_g += P_j V_j     tcgen05.mma with A = P_j read from tensor memory and V as the MN-major B
//                      operand straight from the cache layout [key][dim]
// so P never touches shared memory.  A stream's MMA lane keeps its scores two blocks ahead (its
// first two S first, then P_j V_j followed by S_{j+4}, which overwrites the buffer P_j was read
// from: one thread's MMAs run in the order it issued them): when a stream has stored P_j, the
// scores of its next block are already waiting, so a stream's chain is its own wait - load -
// maximum - exponentials - store and holds no product; the two streams' exponentials and the
// products of both overlap.  The 512 columns of tensor memory: 4 x 64 of scores, 2 x 128 of output.
// Roles in warps of their own: warps 0-3 stream A, warps 4-7 stream B (warp w owns tensor-memory
// lanes 32 (w mod 4) ..), lane 0 of warp 8 feeds Q once and K, lane 0 of warp 10 V, through four-stage
// mbarrier rings by TMA (one box per cache page and 64-column half), lane 0 of warp 9 issues the MMAs
// of stream A and lane 0 of warp 11 those of stream B (12 MMAs per block: with one lane issuing for
// both streams that lane was the bound).
// O_g is rescaled in tensor memory (tcgen05.ld / st) only when a row's maximum has grown by more
// than 8 (in log2 units) beyond the one its p values are taken against: the softmax is the same
// function, p stays below 2^8, and the read-modify-write of O leaves the steady state.
// Keys at positions >= pos0 + R are not part of the prompt: their pages are not fetched, their
// scores are masked and their V rows are zeroed in shared memory before the product (0 x stale
// bits must not produce a NaN).
// Every wait is bounded; on a time-out the kernel records DEV_TIMEOUT in *status, frees its
// tensor memory and returns.
#pragma once
#include "ls_prefill.cuh"

namespace ls {

constexpr int kTcAttnThreads = 384;
constexpr int kTcAttnB = 128;                            // rows per tile, head dim
constexpr int kTcAttnKB = 64;                            // keys per block
constexpr int kTcAttnStages = 4;                         // K and V ring
constexpr int kTcAttnTile = kTcAttnB * kTcAttnB * 2;     // 32 KB: Q, 128 x 128 bf16 as two 64-column halves
constexpr int kTcAttnHalf = kTcAttnTile / 2;
constexpr int kTcAttnStage = kTcAttnKB * kTcAttnB * 2;   // 16 KB: 64 keys x 128 dims as two 64-column halves
constexpr int kTcAttnStageHalf = kTcAttnStage / 2;
constexpr int kTcAttnMaxBoxes = 1024;                    // page boxes of one sequence
constexpr int kTcAttnTmemCols = 512;                     // S_A0 | S_A1 | S_B0 | S_B1 (64 each) | O_A | O_B (128 each)
constexpr size_t kTcAttnSmemBytes = kTcAttnTile + 2 * (size_t)kTcAttnStages * kTcAttnStage + kTcAttnMaxBoxes * 4 +
                                    4 * kTcAttnB * 4 + 1024 + 256;

__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, uint32_t* v)
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
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* v)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]),
          "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]),
          "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]), "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// D[tmem] (+)= A[tmem: 128 lanes x 16 bf16 in 8 columns] * B[smem desc], fp32 accumulate
__device__ __forceinline__ void tc_mma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)  // both roundings (to nearest even) in one instruction
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Shared-memory matrix descriptor of an MN-major operand as the cache holds V ([key][dim], dims
// contiguous): 128-byte rows of 64 dims, 128B-swizzled as TMA wrote them; eight keys are one
// 1024-byte swizzle pattern (stride byte offset: the next eight keys), the next 64 dims are the
// other half of the stage (leading byte offset).
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
    d |= (uint64_t)(kTcAttnStageHalf >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// grid (query heads, tiles of 128 rows), block 384.  q bf16 [R, Hq * 128] (map_q: boxes of 128 rows
// x 64 columns); map_k / map_v: the cache of one layer as rows of 128 dims, row (page * Hkv + kv
// head) * page_size + slot, boxes of box_rows = min(page_size, 64) rows x 64 columns.  Rows at
// positions pos0 .. pos0 + R - 1; keys 0 .. pos0 + R - 1 are in the cache.  The heavy tiles (the
// last rows, which see the most keys) are dealt out first.
__global__ void __launch_bounds__(kTcAttnThreads)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ page_table, int pos0, int R,
                       int Hq, int Hkv, int page_shift, int box_rows, uint16_t* __restrict__ out, int32_t* status)
{
    constexpr int B = kTcAttnB, KB = kTcAttnKB, NS = kTcAttnStages, TILE = kTcAttnTile, HALF = kTcAttnHalf;
    constexpr int STAGE = kTcAttnStage, SHALF = kTcAttnStageHalf;
    extern __shared__ unsigned char tca_raw[];
    const uint32_t raw0 = smem_u32(tca_raw);
    const uint32_t base = (raw0 + 1023u) & ~1023u;  // swizzled tiles want 1024-byte alignment
    unsigned char* gbase = tca_raw + (base - raw0);
    const uint32_t sQ = base, sK = base + TILE, sV = sK + NS * STAGE;
    constexpr int kTiles = TILE + 2 * NS * STAGE;
    int32_t* rowc = reinterpret_cast<int32_t*>(gbase + kTiles);  // first cache row of every page box
    float2* ml = reinterpret_cast<float2*>(gbase + kTiles + kTcAttnMaxBoxes * 4);  // [2][128]: (max, sum) of a stream's row
    const uint32_t bars = base + kTiles + kTcAttnMaxBoxes * 4 + 4 * B * 4;
    auto bar = [&](int i) { return bars + 8u * i; };
    const uint32_t q_full = bar(0);
    auto k_full = [&](int s) { return bar(1 + s); };
    auto k_empty = [&](int s) { return bar(5 + s); };
    auto v_full = [&](int s) { return bar(9 + s); };
    auto v_empty = [&](int s) { return bar(13 + s); };
    auto s_full = [&](int gb) { return bar(17 + gb); };  // gb = 2 * stream + buffer
    // (one per score buffer: a stream may store P into its second buffer before the MMA lane has looked at
    // the first, and a parity wait tells phases apart only while the barrier is at most one phase ahead)
    auto p_full = [&](int gb) { return bar(21 + gb); };
    auto pv_done = [&](int g) { return bar(25 + g); };
    auto all_done = [&](int g) { return bar(27 + g); };
    const uint32_t merge_bar = bar(29), tslot = bar(30);
    __shared__ int failed;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.x, kh = head / (Hq / Hkv);
    const int tile = (int)gridDim.y - 1 - (int)blockIdx.y;
    const int q0 = tile * B;
    const int rows_here = min(B, R - q0);
    const int last_pos = pos0 + q0 + rows_here - 1;
    const int nkb = last_pos / KB + 1;            // key blocks this tile walks
    const int n_valid = pos0 + R;                 // keys in the cache
    const int bpb = KB / box_rows;                // page boxes per key block
    const int nbox = (min(nkb * KB, n_valid) + box_rows - 1) / box_rows;

    if (tid == 0) {
        for (int i = 0; i <= 20; ++i) mbar_init(bar(i), 1);  // q_full, the K and V rings, s_full
        for (int gb = 0; gb < 4; ++gb) mbar_init(p_full(gb), 128);
        mbar_init(pv_done(0), 1);
        mbar_init(pv_done(1), 1);
        mbar_init(all_done(0), 1);
        mbar_init(all_done(1), 1);
        mbar_init(merge_bar, 256);
        failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int e = tid; e < nbox; e += kTcAttnThreads) {
        const int pos = e * box_rows;
        const int page = page_table[pos >> page_shift];
        rowc[e] = ((page * Hkv + kh) << page_shift) + (pos & ((1 << page_shift) - 1));
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tslot), "r"(kTcAttnTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    uint32_t tmem;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem) : "r"(tslot));
    // columns: S_{g,b} at 64 (2 g + b), O_g at 256 + 128 g

    if ((warp == 8 || warp == 10) && lane == 0) {
        // ---------------------------------------------------------------- TMA producers: warp 8 Q and K, warp 10 V
        // (one lane each, so that the next K does not queue behind a V stage that is still being read)
        const bool isK = warp == 8;
        if (isK) {
            mbar_expect_tx(q_full, TILE);
            tma_load_2d(sQ, &map_q, head * B, q0, q_full);
            tma_load_2d(sQ + HALF, &map_q, head * B + 64, q0, q_full);
        }
        const CUtensorMap* map = isK ? &map_k : &map_v;
        const uint32_t ring = isK ? sK : sV;
        for (int j = 0; j < nkb; ++j) {
            const int s = j % NS, key0 = j * KB;
            const int nb = min(bpb, (min(n_valid, key0 + KB) - key0 + box_rows - 1) / box_rows);
            const uint32_t bytes = (uint32_t)nb * box_rows * 256u;
            const uint32_t full = isK ? k_full(s) : v_full(s), empty = isK ? k_empty(s) : v_empty(s);
            if (j >= NS && !mbar_wait(empty, ((j / NS) - 1) & 1)) {
                failed = 1;
                break;
            }
            mbar_expect_tx(full, bytes);
            for (int b = 0; b < nb; ++b) {
                const uint32_t dst = ring + s * STAGE + b * box_rows * 128;
                tma_load_2d(dst, map, 0, rowc[j * bpb + b], full);
                tma_load_2d(dst + SHALF, map, 64, rowc[j * bpb + b], full);
            }
        }
    } else if ((warp == 9 || warp == 11) && lane == 0) {
        // ---------------------------------------------------------------- MMA issuers: warp 9 stream A, warp 11 stream B
        // (the streams share nothing but Q, so each has a lane of its own to issue for it and neither
        // waits behind the other's barriers; one thread's MMAs run in the order it issued them)
        // instruction descriptors: D fp32, A and B bf16, M = 128.  S: N = 64, both operands K-major in
        // shared memory; P V: N = 128, A (= P) in tensor memory, B (= V) MN-major
        const int g = warp == 11;
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KB >> 3) << 17) | ((uint32_t)(B >> 4) << 24);
        const uint32_t idesc_pv =
            (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(B >> 3) << 17) | ((uint32_t)(B >> 4) << 24);
        bool ok = mbar_wait(q_full, 0);
        auto issue_s = [&](int j) {  // S_j into S_{g,b}
            const int s = j % NS, gb = 2 * g + ((j >> 1) & 1);
            if (!mbar_wait(k_full(s), (j / NS) & 1)) return false;
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < B / 16; ++ks) {
                const uint64_t da = umma_desc_sw128(sQ + (ks >> 2) * HALF) + 2 * (ks & 3);
                const uint64_t db = umma_desc_sw128(sK + s * STAGE + (ks >> 2) * SHALF) + 2 * (ks & 3);
                tc_mma_bf16(tmem + gb * KB, da, db, idesc_s, ks != 0);
            }
            tc_commit(k_empty(s));
            tc_commit(s_full(gb));
            return true;
        };
        for (int j = g; j < 4 && j < nkb && ok; j += 2) ok = issue_s(j);
        for (int j = g; j < nkb && ok; j += 2) {
            // O_g += P_j V_j, then S_{j+4} over the buffer P_j was read from
            const int s = j % NS, gb = 2 * g + ((j >> 1) & 1);
            if (!mbar_wait(v_full(s), (j / NS) & 1) || !mbar_wait(p_full(gb), (j >> 2) & 1)) {
                ok = false;
                break;
            }
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < KB / 16; ++kk) {  // 16 keys per MMA: 8 columns of P, 2048 bytes down V
                const uint64_t db = umma_desc_sw128_mn(sV + s * STAGE) + (uint64_t)(kk * (2048 >> 4));
                tc_mma_bf16_ta(tmem + 4 * KB + g * B, tmem + gb * KB + 8 * kk, db, idesc_pv, (j >= 2) || kk != 0);
            }
            tc_commit(v_empty(s));
            tc_commit(pv_done(g));
            if (j + 4 < nkb) ok = issue_s(j + 4);
        }
        if (ok) tc_commit(all_done(g));
        else failed = 1;
    } else if (warp < 8) {
        // ---------------------------------------------------------------- softmax: stream g, one row per thread
        const int w4 = warp & 3, g = warp >> 2, row = w4 * 32 + lane;
        const uint32_t lane0 = tmem + ((uint32_t)(w4 * 32) << 16);
        const uint32_t lane_o = lane0 + 4 * KB + g * B;  // this row of O_g
        const int qpos = min(pos0 + q0 + row, last_pos);  // (rows beyond the prompt: masked like the last one)
        const float sc = rsqrtf((float)B) * 1.4426950408889634f;
        float m_used = -INFINITY, l = 0.f;  // (-inf: no visible key yet; every p so far was zero)
        bool ok = true;
        // (a wait ends for the whole warp alike: the tensor-memory loads below want the warp converged)
        auto wait_all = [&](uint32_t bar_, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(bar_, parity)) != 0; };
        for (int j = g; j < nkb; j += 2) {
            const int i = j >> 1, gb = 2 * g + (i & 1), key0 = j * KB;
            const uint32_t lane_s = lane0 + gb * KB;  // this row of S_{g,b} (and of P)
            if (!wait_all(s_full(gb), (i >> 1) & 1)) {
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t sv[KB];
            tc_ld32_nowait(lane_s, sv);
            tc_ld32_nowait(lane_s + 32, sv + 32);
            tc_wait_ld();
            const int lim = qpos - key0;  // columns 0 .. lim are visible
            if (lim < KB - 1) {
#pragma unroll
                for (int c = 0; c < KB; ++c)
                    if (c > lim) sv[c] = 0xff800000u;  // -inf
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains instead of one of 64
#pragma unroll
            for (int c = 0; c < KB; c += 4) {
#pragma unroll
                for (int k = 0; k < 4; ++k) mx4[k] = fmaxf(mx4[k], __uint_as_float(sv[c + k]));
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;
            const bool first = m_used == -INFINITY;  // nothing accumulated for this row yet: O_g's row is zero (or unwritten)
            const bool need = !first && mx > m_used + 8.f;
            if (__any_sync(0xffffffffu, need)) {  // the warp's 32 rows of O_g, each by its own factor
                // O_g is at rest once the stream's previous product has finished (this block's own is not issued yet)
                if (!wait_all(pv_done(g), (i - 1) & 1)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const float alpha = need ? ex2_approx(m_used - mx) : 1.f;
                l *= alpha;
#pragma unroll 1
                for (int c = 0; c < B / 32; ++c) {
                    uint32_t ov[32];
                    tc_ld32(lane_o + c * 32, ov);
#pragma unroll
                    for (int k = 0; k < 32; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * alpha);
                    tc_st32(lane_o + c * 32, ov);
                }
            }
            if (first || need) m_used = mx;
            // p = exp2(s c - m), rounded to bf16 in place (two per word); the sum takes the unrounded values
            const float neg = m_used == -INFINITY ? 0.f : -m_used;
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < KB / 2; ++c) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(sv[2 * c]), sc, neg));
                const float p1 = ex2_approx(fmaf(__uint_as_float(sv[2 * c + 1]), sc, neg));
                sum4[c & 3] += p0 + p1;
                sv[c] = pack_bf16x2(p0, p1);
            }
            l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            tc_st32(lane_s, sv);
            if (key0 + KB > n_valid) {  // the block reaches beyond the prompt: its V rows there become zeros
                const int s = j % NS;
                if (!wait_all(v_full(s), (j / NS) & 1)) {
                    ok = false;
                    break;
                }
                if (row < KB && row >= n_valid - key0) {
                    const uint32_t vrow = sV + s * STAGE + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vrow + 16 * c), "r"(0u) : "memory");
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vrow + SHALF + 16 * c), "r"(0u) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // V as the tensor core will read it
            }
            tc_fence_before();
            mbar_arrive(p_full(gb));
        }
        // merge the two streams: each thread its row's (max, sum), then columns 64 g .. 64 g + 63 of both outputs
        ml[g * B + row] = make_float2(m_used, l);
        mbar_arrive(merge_bar);
        if (ok && !wait_all(merge_bar, 0)) ok = false;
        if (ok && (!wait_all(all_done(0), 0) || !wait_all(all_done(1), 0))) ok = false;
        tc_fence_after();
        if (ok) {
            const float2 a = ml[row], b = ml[B + row];  // (stream A has seen key 0: its maximum is finite)
            const bool hasB = nkb > 1 && b.x != -INFINITY;
            const float m = hasB ? fmaxf(a.x, b.x) : a.x;
            const float wa = ex2_approx(a.x - m), wb = hasB ? ex2_approx(b.x - m) : 0.f;
            const float inv = 1.f / (a.y * wa + b.y * wb);
            const float fa = wa * inv, fb = wb * inv;
            const uint32_t oa = lane0 + 4 * KB + 64 * g, ob = oa + B;
            uint16_t* dst = out + ((size_t)(q0 + row) * Hq + head) * B + 64 * g;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                uint32_t va[32], vb[32];
                tc_ld32_nowait(oa + c * 32, va);
                if (nkb > 1) tc_ld32_nowait(ob + c * 32, vb);
                tc_wait_ld();
                if (row < rows_here) {
#pragma unroll
                    for (int k = 0; k < 32; k += 8) {
                        float o[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            o[e] = __uint_as_float(va[k + e]) * fa;
                            if (hasB) o[e] = fmaf(__uint_as_float(vb[k + e]), fb, o[e]);
                        }
                        uint4 w;
                        w.x = pack_bf16x2(o[0], o[1]);
                        w.y = pack_bf16x2(o[2], o[3]);
                        w.z = pack_bf16x2(o[4], o[5]);
                        w.w = pack_bf16x2(o[6], o[7]);
                        *reinterpret_cast<uint4*>(dst + c * 32 + k) = w;
                    }
                }
            }
        } else {
            failed = 1;
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (failed && tid == 0) {
        if (status) *status = DEV_TIMEOUT;
        __nanosleep(1000000);  // let copies that may still be in flight land before the CTA goes away
    }
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcAttnTmemCols) : "memory");
}

}  // namespace ls

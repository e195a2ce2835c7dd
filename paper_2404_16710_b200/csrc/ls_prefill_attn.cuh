// Causal attention of the prompt pass on the 5th-gen tensor cores (head dim 128).
//
// One CTA per (tile of 128 prompt rows, query head) walks the key blocks of 128 cache positions
// that its rows can see, as TWO independent online-softmax streams: stream A takes the even
// blocks, stream B the odd ones, each with its own score buffer, running (max, sum) per row and
// output accumulator; the two are merged at the end like the spans of a split cache.  While one
// stream's four warps are in their latency chain (wait for the scores, tcgen05.ld, maximum, 128
// exponentials per row, store) the other stream's products run on the tensor pipe, and the
// exponentials of the two streams keep the special-function unit busy in turn.  Per block j of
// stream g = j mod 2:
//   S_j = Q K_j^T      tcgen05.mma, 128 x 128 x 128, fp32 into S_g (tensor memory)
//   P_j = exp2(S_j c - m)   four warps, one query row per thread: the row of S_g by tcgen05.ld,
//                      running maximum m and sum l in registers, P_j rounded to bf16 and written
//                      back by tcgen05.st over the first 64 columns of S_g (two keys per word)
//   O_g += P_j V_j     tcgen05.mma with A = P_j read from tensor memory and V as the MN-major B
//                      operand straight from the cache layout [key][dim]
// so P never touches shared memory.  S_{j+2} overwrites P_j: it is issued after P_j V_j and the
// tensor pipe runs its instructions in order.
// Roles in warps of their own: warps 0-3 stream A, warps 4-7 stream B (warp w owns tensor-memory
// lanes 32 (w mod 4) ..), lane 0 of warp 8 feeds Q once and K, lane 0 of warp 10 V, through two-stage
// mbarrier rings by TMA (one box per cache page and 64-column half; stage = stream), lane 0 of
// warp 9 issues the MMAs in the order S_0, S_1, PV_0, S_2, PV_1, S_3, ...
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

constexpr int kTcAttnThreads = 352;
constexpr int kTcAttnB = 128;                            // rows per tile, keys per block, head dim
constexpr int kTcAttnTile = kTcAttnB * kTcAttnB * 2;     // 32 KB: 128 x 128 bf16 as two 64-column halves
constexpr int kTcAttnHalf = kTcAttnTile / 2;
constexpr int kTcAttnMaxBoxes = 1024;                    // page boxes of one sequence
constexpr int kTcAttnTmemCols = 512;                     // S_A | S_B | O_A | O_B
constexpr size_t kTcAttnSmemBytes = 5 * (size_t)kTcAttnTile + kTcAttnMaxBoxes * 4 + 4 * kTcAttnB * 4 + 1024 + 256;

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
// other half of the tile (leading byte offset).
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
    d |= (uint64_t)(kTcAttnHalf >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// grid (query heads, tiles of 128 rows), block 352.  q bf16 [R, Hq * 128] (map_q: boxes of 128 rows
// x 64 columns); map_k / map_v: the cache of one layer as rows of 128 dims, row (page * Hkv + kv
// head) * page_size + slot, boxes of box_rows = min(page_size, 128) rows x 64 columns.  Rows at
// positions pos0 .. pos0 + R - 1; keys 0 .. pos0 + R - 1 are in the cache.  The heavy tiles (the
// last rows, which see the most keys) are dealt out first.
__global__ void __launch_bounds__(kTcAttnThreads)
prefill_attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ page_table, int pos0, int R,
                       int Hq, int Hkv, int page_shift, int box_rows, uint16_t* __restrict__ out, int32_t* status)
{
    constexpr int B = kTcAttnB, TILE = kTcAttnTile, HALF = kTcAttnHalf;
    extern __shared__ unsigned char tca_raw[];
    const uint32_t raw0 = smem_u32(tca_raw);
    const uint32_t base = (raw0 + 1023u) & ~1023u;  // swizzled tiles want 1024-byte alignment
    unsigned char* gbase = tca_raw + (base - raw0);
    const uint32_t sQ = base, sK = base + TILE, sV = base + 3 * TILE;
    int32_t* rowc = reinterpret_cast<int32_t*>(gbase + 5 * TILE);  // first cache row of every page box
    float2* ml = reinterpret_cast<float2*>(gbase + 5 * TILE + kTcAttnMaxBoxes * 4);  // [2][128]: (max, sum) of a stream's row
    const uint32_t bars = base + 5 * TILE + kTcAttnMaxBoxes * 4 + 4 * B * 4;
    const uint32_t q_full = bars;
    auto k_full = [&](int s) { return bars + 8u + 8u * s; };
    auto k_empty = [&](int s) { return bars + 24u + 8u * s; };
    auto v_full = [&](int s) { return bars + 40u + 8u * s; };
    auto v_empty = [&](int s) { return bars + 56u + 8u * s; };
    auto s_full = [&](int s) { return bars + 72u + 8u * s; };
    auto p_full = [&](int s) { return bars + 88u + 8u * s; };
    const uint32_t all_done = bars + 104u, merge_bar = bars + 112u, tslot = bars + 120u;
    __shared__ int failed;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.x, kh = head / (Hq / Hkv);
    const int tile = (int)gridDim.y - 1 - (int)blockIdx.y;
    const int q0 = tile * B;
    const int rows_here = min(B, R - q0);
    const int last_pos = pos0 + q0 + rows_here - 1;
    const int nkb = last_pos / B + 1;             // key blocks this tile walks
    const int n_valid = pos0 + R;                 // keys in the cache
    const int bpb = B / box_rows;                 // page boxes per key block
    const int nbox = (min(nkb * B, n_valid) + box_rows - 1) / box_rows;

    if (tid == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(k_full(s), 1);
            mbar_init(k_empty(s), 1);
            mbar_init(v_full(s), 1);
            mbar_init(v_empty(s), 1);
            mbar_init(s_full(s), 1);
            mbar_init(p_full(s), 128);
        }
        mbar_init(all_done, 1);
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
    // columns: S_A 0.., S_B 128.., O_A 256.., O_B 384..

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
            const int s = j & 1, key0 = j * B;
            const int nb = min(bpb, (min(n_valid, key0 + B) - key0 + box_rows - 1) / box_rows);
            const uint32_t bytes = (uint32_t)nb * box_rows * 256u;
            const uint32_t full = isK ? k_full(s) : v_full(s), empty = isK ? k_empty(s) : v_empty(s);
            if (j >= 2 && !mbar_wait(empty, ((j >> 1) - 1) & 1)) {
                failed = 1;
                break;
            }
            mbar_expect_tx(full, bytes);
            for (int b = 0; b < nb; ++b) {
                const uint32_t dst = ring + s * TILE + b * box_rows * 128;
                tma_load_2d(dst, map, 0, rowc[j * bpb + b], full);
                tma_load_2d(dst + HALF, map, 64, rowc[j * bpb + b], full);
            }
        }
    } else if (warp == 9 && lane == 0) {
        // ---------------------------------------------------------------- MMA issuer
        // instruction descriptors: D fp32, A and B bf16, N = 128, M = 128; S: both operands K-major
        // in shared memory; P V: A (= P) in tensor memory, B (= V) MN-major
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(B >> 3) << 17) | ((uint32_t)(B >> 4) << 24);
        const uint32_t idesc_pv = idesc_s | (1u << 16);
        bool ok = mbar_wait(q_full, 0);
        for (int j = 0; j <= nkb && ok; ++j) {
            if (j < nkb) {  // S_j into S_g (behind P_{j-2} V_{j-2} on the pipe, which read P from the same columns)
                const int g = j & 1;
                if (!mbar_wait(k_full(g), (j >> 1) & 1)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < B / 16; ++ks) {
                    const uint64_t da = umma_desc_sw128(sQ + (ks >> 2) * HALF) + 2 * (ks & 3);
                    const uint64_t db = umma_desc_sw128(sK + g * TILE + (ks >> 2) * HALF) + 2 * (ks & 3);
                    tc_mma_bf16(tmem + g * B, da, db, idesc_s, ks != 0);
                }
                tc_commit(k_empty(g));
                tc_commit(s_full(g));
            }
            if (j >= 1) {  // O_g += P_{j-1} V_{j-1}
                const int jj = j - 1, g = jj & 1;
                if (!mbar_wait(v_full(g), (jj >> 1) & 1) || !mbar_wait(p_full(g), (jj >> 1) & 1)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < B / 16; ++kk) {  // 16 keys per MMA: 8 columns of P, 2048 bytes down V
                    const uint64_t db = umma_desc_sw128_mn(sV + g * TILE) + (uint64_t)(kk * (2048 >> 4));
                    tc_mma_bf16_ta(tmem + (2 + g) * B, tmem + g * B + 8 * kk, db, idesc_pv, (jj >= 2) || kk != 0);
                }
                tc_commit(v_empty(g));
            }
        }
        if (ok) tc_commit(all_done);
        else failed = 1;
    } else if (warp < 8) {
        // ---------------------------------------------------------------- softmax: stream g, one row per thread
        const int w4 = warp & 3, g = warp >> 2, row = w4 * 32 + lane;
        const uint32_t lane_s = tmem + ((uint32_t)(w4 * 32) << 16) + g * B;        // this row of S_g (and P)
        const uint32_t lane_o = tmem + ((uint32_t)(w4 * 32) << 16) + (2 + g) * B;  // this row of O_g
        const int qpos = min(pos0 + q0 + row, last_pos);  // (rows beyond the prompt: masked like the last one)
        const float sc = rsqrtf((float)B) * 1.4426950408889634f;
        float m_used = -INFINITY, l = 0.f;  // (-inf: no visible key yet; every p so far was zero)
        bool ok = true;
        // (a wait ends for the whole warp alike: the tensor-memory loads below want the warp converged)
        auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(bar, parity)) != 0; };
        for (int j = g; j < nkb; j += 2) {
            const int i = j >> 1, key0 = j * B;
            // (S_j complete means P_{j-2} V_{j-2} complete: the commit covers everything issued before it)
            if (!wait_all(s_full(g), i & 1)) {
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t sv[B];
#pragma unroll
            for (int c = 0; c < B / 32; ++c) tc_ld32_nowait(lane_s + c * 32, sv + 32 * c);
            tc_wait_ld();
            const int lim = qpos - key0;  // columns 0 .. lim are visible
            if (lim < B - 1) {
#pragma unroll
                for (int c = 0; c < B; ++c)
                    if (c > lim) sv[c] = 0xff800000u;  // -inf
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains instead of one of 128
#pragma unroll
            for (int c = 0; c < B; c += 4) {
#pragma unroll
                for (int k = 0; k < 4; ++k) mx4[k] = fmaxf(mx4[k], __uint_as_float(sv[c + k]));
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;
            const bool first = m_used == -INFINITY;  // nothing accumulated for this row yet: O_g's row is zero (or unwritten)
            const bool need = !first && mx > m_used + 8.f;
            if (__any_sync(0xffffffffu, need)) {  // the warp's 32 rows of O_g, each by its own factor
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
            for (int c = 0; c < B / 2; ++c) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(sv[2 * c]), sc, neg));
                const float p1 = ex2_approx(fmaf(__uint_as_float(sv[2 * c + 1]), sc, neg));
                sum4[c & 3] += p0 + p1;
                sv[c] = pack_bf16x2(p0, p1);
            }
            l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            tc_st32(lane_s, sv);
            tc_st32(lane_s + 32, sv + 32);
            if (key0 + B > n_valid) {  // the block reaches beyond the prompt: its V rows there become zeros
                if (!wait_all(v_full(g), i & 1)) {
                    ok = false;
                    break;
                }
                if (row >= n_valid - key0) {
                    const uint32_t vrow = sV + g * TILE + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vrow + 16 * c), "r"(0u) : "memory");
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vrow + HALF + 16 * c), "r"(0u) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // V as the tensor core will read it
            }
            tc_fence_before();
            mbar_arrive(p_full(g));
        }
        // merge the two streams: each thread its row's (max, sum), then columns 64 g .. 64 g + 63 of both outputs
        ml[g * B + row] = make_float2(m_used, l);
        mbar_arrive(merge_bar);
        if (ok && !wait_all(merge_bar, 0)) ok = false;
        if (ok && !wait_all(all_done, 0)) ok = false;
        tc_fence_after();
        if (ok) {
            const float2 a = ml[row], b = ml[B + row];  // (stream A has seen key 0: its maximum is finite)
            const bool hasB = nkb > 1 && b.x != -INFINITY;
            const float m = hasB ? fmaxf(a.x, b.x) : a.x;
            const float wa = ex2_approx(a.x - m), wb = hasB ? ex2_approx(b.x - m) : 0.f;
            const float inv = 1.f / (a.y * wa + b.y * wb);
            const float fa = wa * inv, fb = wb * inv;
            const uint32_t oa = tmem + ((uint32_t)(w4 * 32) << 16) + 2 * B + 64 * g, ob = oa + B;
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

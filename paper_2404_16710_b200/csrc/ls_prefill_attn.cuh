// Causal attention of the prompt pass on the 5th-gen tensor cores (head dim 128).
//
// One CTA per (tile of 128 prompt rows, query head) walks the key blocks of 128 cache positions
// that its rows can see.  Per key block j:
//   S_j = Q K_j^T      tcgen05.mma, 128 x 128 x 128, fp32 in tensor memory (two S buffers)
//   P_j = exp2(S_j c - m)   eight warps, two threads per query row (64 columns each): tcgen05.ld of
//                      the row, running maximum m and sum l in registers, P_j rounded to bf16 into
//                      128B-swizzled shared memory (the K-major A operand of the next product)
//   O  += P_j V_j      tcgen05.mma with V as the MN-major B operand straight from the cache
//                      layout [key][dim]; O stays in tensor memory for the whole walk
// Roles in warps of their own: warps 0-7 softmax and epilogue (warps w and w + 4 own tensor-memory
// lanes 32w..32w+31), lane 0 of warp 8 feeds Q once and K, lane 0
// of warp 10 V, through two-stage mbarrier rings by TMA (one box per cache page and 64-column half),
// lane 0 of warp 9 issues the MMAs.  S_{j+1} is issued before the MMA lane waits for P_j, so the tensor pipe
// works on it while the softmax warps are busy with block j.
// O is rescaled in tensor memory (tcgen05.ld / st) only when a row's maximum has grown by more
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
constexpr int kTcAttnTmemCols = 512;                     // S0 | S1 | O | (unused)
constexpr size_t kTcAttnSmemBytes = 6 * (size_t)kTcAttnTile + kTcAttnMaxBoxes * 4 + 4 * kTcAttnB * 4 + 1024 + 256;

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
    const uint32_t sQ = base, sK = base + TILE, sV = base + 3 * TILE, sP = base + 5 * TILE;
    int32_t* rowc = reinterpret_cast<int32_t*>(gbase + 6 * TILE);  // first cache row of every page box
    float* xch = reinterpret_cast<float*>(gbase + 6 * TILE + kTcAttnMaxBoxes * 4);  // [2][2][128]: what the two threads of a row swap
    const uint32_t bars = base + 6 * TILE + kTcAttnMaxBoxes * 4 + 4 * B * 4;
    const uint32_t q_full = bars;
    auto k_full = [&](int s) { return bars + 8u + 8u * s; };
    auto k_empty = [&](int s) { return bars + 24u + 8u * s; };
    auto v_full = [&](int s) { return bars + 40u + 8u * s; };
    auto v_empty = [&](int s) { return bars + 56u + 8u * s; };
    auto s_full = [&](int s) { return bars + 72u + 8u * s; };
    const uint32_t p_full = bars + 88u, pv_done = bars + 96u, tslot = bars + 104u;
    auto pair_bar = [&](int w) { return bars + 112u + 8u * w; };
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
        }
        mbar_init(p_full, 256);
        mbar_init(pv_done, 1);
        for (int w = 0; w < 4; ++w) mbar_init(pair_bar(w), 64);
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
    const uint32_t tO = tmem + 2 * B;

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
        // instruction descriptors: D fp32, A and B bf16, N = 128, M = 128; S: both operands K-major,
        // P V: B (= V) MN-major
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(B >> 3) << 17) | ((uint32_t)(B >> 4) << 24);
        const uint32_t idesc_pv = idesc_s | (1u << 16);
        bool ok = mbar_wait(q_full, 0);
        auto issue_s = [&](int j) {  // S_j into buffer j & 1
            const int s = j & 1;
            if (!mbar_wait(k_full(s), (j >> 1) & 1)) return false;
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < B / 16; ++ks) {
                const uint64_t da = umma_desc_sw128(sQ + (ks >> 2) * HALF) + 2 * (ks & 3);
                const uint64_t db = umma_desc_sw128(sK + s * TILE + (ks >> 2) * HALF) + 2 * (ks & 3);
                tc_mma_bf16(tmem + s * B, da, db, idesc_s, ks != 0);
            }
            tc_commit(k_empty(s));
            tc_commit(s_full(s));
            return true;
        };
        ok = ok && issue_s(0);
        for (int j = 0; j < nkb && ok; ++j) {
            // (buffer (j + 1) & 1 was last read for block j - 1, whose P has been waited for)
            if (j + 1 < nkb && !issue_s(j + 1)) {
                ok = false;
                break;
            }
            const int s = j & 1;
            if (!mbar_wait(v_full(s), (j >> 1) & 1) || !mbar_wait(p_full, j & 1)) {
                ok = false;
                break;
            }
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < B / 16; ++kk) {  // 16 keys per MMA: 32 bytes along P's rows, 2048 bytes down V
                const uint64_t da = umma_desc_sw128(sP + (kk >> 2) * HALF) + 2 * (kk & 3);
                const uint64_t db = umma_desc_sw128_mn(sV + s * TILE) + (uint64_t)(kk * (2048 >> 4));
                tc_mma_bf16(tO, da, db, idesc_pv, (j | kk) != 0);
            }
            tc_commit(v_empty(s));
            tc_commit(pv_done);
        }
        if (!ok) failed = 1;
    } else if (warp < 8) {
        // ---------------------------------------------------------------- softmax, two threads per row
        // warps w and w + 4 own tensor-memory lanes 32 (w % 4) ..: thread (row, half) takes columns
        // 64 half .. 64 half + 63 of its row of S (and of O); the two meet once per block to agree on
        // the row's maximum (an mbarrier per pair of warps, so that this wait is bounded like the others)
        const int w4 = warp & 3, half = warp >> 2, row = w4 * 32 + lane;
        const uint32_t lane_t = tmem + ((uint32_t)(w4 * 32) << 16) + 64 * half;
        const uint32_t lane_o = tO + ((uint32_t)(w4 * 32) << 16) + 64 * half;
        const int qpos = min(pos0 + q0 + row, last_pos);  // (rows beyond the prompt: masked like the last one)
        const float sc = rsqrtf((float)B) * 1.4426950408889634f;
        float m_used = 0.f, l = 0.f;
        bool ok = true;
        // (a wait ends for the whole warp alike: the tensor-memory loads below want the warp converged)
        auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(bar, parity)) != 0; };
        int n_meet = 0;
        // hand v to the row's other thread and return what that one handed over
        auto swap_with_partner = [&](float v, float& other) {
            float* slot = xch + (n_meet & 1) * 2 * B;
            slot[half * B + row] = v;
            mbar_arrive(pair_bar(w4));
            if (!wait_all(pair_bar(w4), n_meet & 1)) return false;
            other = slot[(half ^ 1) * B + row];
            ++n_meet;
            return true;
        };
        for (int j = 0; j < nkb; ++j) {
            const int s = j & 1, key0 = j * B;
            if (!wait_all(s_full(s), (j >> 1) & 1)) {
                ok = false;
                break;
            }
            tc_fence_after();
            uint32_t sv[B / 2];
            tc_ld32_nowait(lane_t + s * B, sv);
            tc_ld32_nowait(lane_t + s * B + 32, sv + 32);
            tc_wait_ld();
            const int lim = qpos - key0 - 64 * half;  // this thread's columns 0 .. lim are visible
            if (lim < B / 2 - 1) {
#pragma unroll
                for (int c = 0; c < B / 2; ++c)
                    if (c > lim) sv[c] = 0xff800000u;  // -inf
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four chains instead of one
#pragma unroll
            for (int c = 0; c < B / 2; c += 4) {
#pragma unroll
                for (int i = 0; i < 4; ++i) mx4[i] = fmaxf(mx4[i], __uint_as_float(sv[c + i]));
            }
            float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc, mx_other;
            if (!swap_with_partner(mx, mx_other)) {
                ok = false;
                break;
            }
            mx = fmaxf(mx, mx_other);
            if (j == 0) {
                m_used = mx;  // key 0 is visible to every row
            } else {
                const bool need = mx > m_used + 8.f;
                if (__any_sync(0xffffffffu, need)) {  // the warp's 32 rows of O, each by its own factor
                    if (!wait_all(pv_done, (j - 1) & 1)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const float alpha = need ? ex2_approx(m_used - mx) : 1.f;
                    if (need) m_used = mx;
                    l *= alpha;
#pragma unroll 1
                    for (int c = 0; c < 2; ++c) {
                        uint32_t ov[32];
                        tc_ld32(lane_o + c * 32, ov);
#pragma unroll
                        for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                        tc_st32(lane_o + c * 32, ov);
                    }
                }
            }
            // p = exp2(s c - m), rounded to bf16 in place (two per word); the sum takes the unrounded values
            const float neg = -m_used;
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < B / 4; ++c) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(sv[2 * c]), sc, neg));
                const float p1 = ex2_approx(fmaf(__uint_as_float(sv[2 * c + 1]), sc, neg));
                sum4[c & 3] += p0 + p1;
                sv[c] = pack_bf16x2(p0, p1);
            }
            l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            // P's buffer is free (and O at rest) once the product of block j - 1 has finished
            if (j > 0 && !wait_all(pv_done, (j - 1) & 1)) {
                ok = false;
                break;
            }
            {
                const uint32_t prow = sP + half * HALF + row * 128;
#pragma unroll
                for (int c16 = 0; c16 < 8; ++c16) {
                    const uint32_t addr = prow + ((c16 ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(sv[4 * c16]), "r"(sv[4 * c16 + 1]),
                                 "r"(sv[4 * c16 + 2]), "r"(sv[4 * c16 + 3])
                                 : "memory");
                }
            }
            if (key0 + B > n_valid) {  // the block reaches beyond the prompt: its V rows there become zeros
                if (!wait_all(v_full(s), (j >> 1) & 1)) {
                    ok = false;
                    break;
                }
                if (row >= n_valid - key0) {
                    const uint32_t vrow = sV + s * TILE + half * HALF + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vrow + 16 * c), "r"(0u) : "memory");
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // P (and V) as the tensor core will read them
            tc_fence_before();
            mbar_arrive(p_full);
        }
        float l_other = 0.f;
        if (ok && !swap_with_partner(l, l_other)) ok = false;
        if (ok && !wait_all(pv_done, (nkb - 1) & 1)) ok = false;
        tc_fence_after();
        if (ok) {
            const float inv = 1.f / (l + l_other);
            uint16_t* dst = out + ((size_t)(q0 + row) * Hq + head) * B + 64 * half;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                uint32_t ov[32];
                tc_ld32(lane_o + c * 32, ov);
                if (row < rows_here) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(ov[i]) * inv, __uint_as_float(ov[i + 1]) * inv);
                        w.y = pack_bf16x2(__uint_as_float(ov[i + 2]) * inv, __uint_as_float(ov[i + 3]) * inv);
                        w.z = pack_bf16x2(__uint_as_float(ov[i + 4]) * inv, __uint_as_float(ov[i + 5]) * inv);
                        w.w = pack_bf16x2(__uint_as_float(ov[i + 6]) * inv, __uint_as_float(ov[i + 7]) * inv);
                        *reinterpret_cast<uint4*>(dst + c * 32 + i) = w;
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

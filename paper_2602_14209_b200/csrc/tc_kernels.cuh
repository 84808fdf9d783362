// Tensor-core (tcgen05 + TMEM + TMA) kernels of the path for sm_100a.
//
// Warp roles in every kernel here: warps 0-3 and 4-7 are two "softmax" warpgroups (warp w owns TMEM lanes
// 32*(w%4)..+31), one producer warp issues TMA tile loads, one warp issues tcgen05.mma from a single lane and
// owns the TMEM allocation.  All hand-offs go through mbarriers with bounded waits (sm100_ptx.cuh).
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mage {
namespace tc {

constexpr int kTile = 128;                 // keys per tile
constexpr int kBoxBytes = 64 * 128;        // one TMA box: 64 rows x 64 bf16 (128 bytes), 128-byte swizzled
constexpr int kHalfBytes = kTile * 128;    // 128 rows x 128 bytes: one d-half of a K or V tile
constexpr int kTileBytes = 2 * kHalfBytes; // 32 KB

// Coordinates (c1, c2, c3) of the 64-row TMA box that starts at logical cache position j (a multiple of 64).
// Positions at or beyond N map to an out-of-range box, which TMA fills with zeros.
__device__ __forceinline__ void cache_box_coords(const KvView &kv, int p, int h, int j, int N, int &c1, int &c2, int &c3,
                                                 unsigned *status) {
    if (kv.page_size == 0) {
        c1 = j < N ? j : kv.N_max + 64;
        c2 = h;
        c3 = p;
        return;
    }
    c1 = j % kv.page_size;
    c2 = h;
    c3 = kv.num_pages;                     // out of range: zero fill
    if (j < N) {
        const int page = kv.block_table[(long long)p * kv.max_pages + j / kv.page_size];
        if (page >= 0 && page < kv.num_pages) c3 = page;
        else if (status) atomicOr(status, MAGE_DEV_BAD_PAGE);
    }
}

// ------------------------------------------------------------------------------------------------------------
// Block-score kernel (Eq. 4): score[j] = 1/M * sum_r exp2(scale_log2 * <q_r, k_j> - lse2_r).
// Orientation: keys are the MMA M dimension (TMEM lanes), query rows the N dimension (TMEM columns), so each
// thread owns one key and its sum over rows needs no cross-thread reduction.  One CTA walks `tiles_per_cta`
// consecutive 128-key tiles of one KV head; S^T tiles are double-buffered in TMEM, one buffer per warpgroup.
// ------------------------------------------------------------------------------------------------------------
constexpr int kScoreStages = 4;
constexpr int kScoreThreads = 320;
constexpr int kScoreQBytes = 2 * 256 * 128;           // up to 256 query rows, two d-halves
constexpr size_t kScoreSmemBytes = 1024 + kScoreQBytes + kScoreStages * kTileBytes + 256 * sizeof(float) + 256;

__global__ void __launch_bounds__(kScoreThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, KvView kv, Plan plan,
             int row_begin, int rows, int tiles_per_cta, float scale_log2, const float *__restrict__ ws,
             float *__restrict__ scores, int accumulate, unsigned *status) {
    using namespace ptx;
    const int z = blockIdx.y, p = z / kv.H_kv, h = z % kv.H_kv;
    const int N = seq_len_of(kv, p);
    const int tiles_total = (N + kTile - 1) / kTile;
    const int tile0 = blockIdx.x * tiles_per_cta;
    if (tile0 >= tiles_total) return;
    const int n_my = min(tiles_per_cta, tiles_total - tile0);

    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *q_s = base, *k_s = base + kScoreQBytes;
    float *neg_lse_s = reinterpret_cast<float *>(k_s + kScoreStages * kTileBytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(neg_lse_s + 256);
    // barrier indices
    enum { Q_FULL = 0, FULL = 1, EMPTY = FULL + kScoreStages, T_FULL = EMPTY + kScoreStages, T_EMPTY = T_FULL + 2, N_BARS = T_EMPTY + 2 };
    uint32_t *tmem_ptr_s = reinterpret_cast<uint32_t *>(bars + N_BARS);
    volatile int *abort_s = reinterpret_cast<volatile int *>(tmem_ptr_s + 1);
    auto bar = [&](int i) { return smem_u32(bars + i); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rows64 = (rows + 63) & ~63, n_mma = (rows + 15) & ~15;

    if (tid == 0) {
        *abort_s = 0;
        mbar_init(bar(Q_FULL), 1);
        for (int s = 0; s < kScoreStages; ++s) { mbar_init(bar(FULL + s), 1); mbar_init(bar(EMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar(T_FULL + b), 1); mbar_init(bar(T_EMPTY + b), 128); }
        fence_mbar_init();
    }
    if (warp == 9) { tmem_alloc(smem_u32(tmem_ptr_s), 512); tmem_relinquish(); }
    if (tid < 256) neg_lse_s[tid] = tid < rows ? ws[plan.off_neg_lse + (size_t)z * plan.Mw + row_begin + tid] : 0.f;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_s;

    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            const int q_row0 = (p * kv.H_q + h * kv.G) * kv.B + row_begin;
            mbar_arrive_expect_tx(bar(Q_FULL), 2 * rows64 * 128);
            for (int dh = 0; dh < 2; ++dh)
                for (int rb = 0; rb < rows64 / 64; ++rb)
                    tma_load_2d(smem_u32(q_s + dh * (kScoreQBytes / 2) + rb * kBoxBytes), &map_q, bar(Q_FULL), dh * 64, q_row0 + rb * 64);
            int issued = 0;
            for (int i = 0; i < n_my; ++i) {
                const int slot = i % kScoreStages, u = i / kScoreStages;
                if (!mbar_wait(bar(EMPTY + slot), (u & 1) ^ 1, abort_s, status)) break;
                mbar_arrive_expect_tx(bar(FULL + slot), kTileBytes);
                const int j0 = (tile0 + i) * kTile;
                for (int kh = 0; kh < 2; ++kh) {
                    int c1, c2, c3;
                    cache_box_coords(kv, p, h, j0 + kh * 64, N, c1, c2, c3, status);
                    for (int dh = 0; dh < 2; ++dh)
                        tma_load_4d(smem_u32(k_s + slot * kTileBytes + dh * kHalfBytes + kh * kBoxBytes), &map_k, bar(FULL + slot), dh * 64, c1, c2, c3);
                }
                issued = i + 1;
            }
            if (*abort_s) {   // give the copies already in flight a bounded chance to land before the CTA exits
                for (int i = max(0, issued - kScoreStages); i < issued; ++i) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(bar(FULL + i % kScoreStages), (i / kScoreStages) & 1) && clock64() - t0 < 2000000) {}
                }
            }
        }
    } else if (warp == 9) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16_f32(n_mma, false, false);
            bool ok = mbar_wait(bar(Q_FULL), 0, abort_s, status);
            for (int i = 0; ok && i < n_my; ++i) {
                const int slot = i % kScoreStages, u = i / kScoreStages, buf = i & 1, ub = i >> 1;
                if (!mbar_wait(bar(T_EMPTY + buf), (ub & 1) ^ 1, abort_s, status)) break;
                if (!mbar_wait(bar(FULL + slot), u & 1, abort_s, status)) break;
                tc_fence_after_sync();
                const uint32_t k_addr = smem_u32(k_s + slot * kTileBytes), q_addr = smem_u32(q_s);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a = smem_desc_sw128(k_addr + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024);
                    const uint64_t b = smem_desc_sw128(q_addr + (ks >> 2) * (kScoreQBytes / 2) + (ks & 3) * 32, 16, 1024);
                    umma_ss(tmem_base + buf * 256, a, b, idesc, ks > 0);
                }
                umma_commit(bar(EMPTY + slot));
                umma_commit(bar(T_FULL + buf));
            }
        }
    } else {
        const int wg = warp >> 2, w4 = warp & 3;
        const float inv_m = 1.f / (float)kv.M;
        float *srow = scores + (size_t)z * kv.N_max;
        for (int i = wg; i < n_my; i += 2) {
            const int ub = i >> 1;
            if (!__all_sync(0xffffffffu, mbar_wait(bar(T_FULL + wg), ub & 1, abort_s, status))) break;
            tc_fence_after_sync();
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t taddr = tmem_base + wg * 256 + ((uint32_t)(w4 * 32) << 16);
            for (int c0 = 0; c0 < rows; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(taddr + c0, r);
                tmem_wait_ld();
                if (c0 + 32 <= rows) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) acc[e & 3] += ex2(fmaf(__uint_as_float(r[e]), scale_log2, neg_lse_s[c0 + e]));
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c0 + e < rows) acc[e & 3] += ex2(fmaf(__uint_as_float(r[e]), scale_log2, neg_lse_s[c0 + e]));
                }
            }
            tc_fence_before_sync();
            mbar_arrive(bar(T_EMPTY + wg));
            const int j = (tile0 + i) * kTile + w4 * 32 + lane;
            if (j < N) {
                const float v = ((acc[0] + acc[1]) + (acc[2] + acc[3])) * inv_m;
                srow[j] = accumulate ? srow[j] + v : v;
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

}  // namespace tc
}  // namespace mage

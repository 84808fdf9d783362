// Tensor-core (tcgen05 + TMEM + TMA) kernels of the path for sm_100a.
//
// Warp roles in every kernel here: the first warps form "softmax" warpgroups of four warps (warp w owns TMEM lanes
// 32*(w%4)..+31: two warpgroups in the attention kernel, four in the score kernel), then come the producer warp(s)
// that issue TMA tile loads or gather rows with cp.async, and one warp that issues tcgen05.mma from a single lane
// and owns the TMEM allocation.  All hand-offs go through mbarriers with bounded waits (sm100_ptx.cuh).
#pragma once
#include <type_traits>
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "k8.cuh"

namespace mage {
namespace tc {

// Development aid, compiled out of the library: with -DMAGE_TIMING, CTA (0,0,0) of the attention kernel writes
// %globaltimer stamps at its hand-off points into a device array that mage_debug_stamps() copies out.
#ifdef MAGE_TIMING
__device__ unsigned long long g_stamps[128];
__device__ __forceinline__ void stamp_at(int i) {
    if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && i < 100) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_stamps[i] = t;
    }
}
#define MAGE_STAMP(i) stamp_at(i)
#define MAGE_CLK(i) do { if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) g_stamps[i] = (unsigned long long)clock64(); } while (0)
#else
#define MAGE_STAMP(i) ((void)0)
#define MAGE_CLK(i) ((void)0)
#endif

constexpr int kTile = 128;                 // keys per tile
constexpr int kBoxBytes = 64 * 128;        // one TMA box: 64 rows x 64 bf16 (128 bytes), 128-byte swizzled
constexpr int kHalfBytes = kTile * 128;    // 128 rows x 128 bytes: one d-half of a K or V tile
constexpr int kTileBytes = 2 * kHalfBytes; // 32 KB

// Coordinates (c1, c2, c3) of the 64-row TMA box that starts at logical cache position j (a multiple of 64).
// Positions at or beyond N map to an out-of-range box, which TMA fills with zeros.  Returns true when the box lies
// inside the prefix but its page id is out of range: the box is zero-filled too, the status bit is raised, and the
// caller has to leave its 64 keys out of the softmax (a skipped key is not a key with logit 0).
__device__ __forceinline__ bool cache_box_coords(const KvView &kv, int p, int h, int j, int N, int &c1, int &c2, int &c3,
                                                 unsigned *status) {
    if (kv.page_size == 0) {
        c1 = j < N ? j : kv.N_max + 64;
        c2 = h;
        c3 = p;
        return false;
    }
    c1 = j % kv.page_size;
    c2 = h;
    c3 = kv.num_pages;                     // out of range: zero fill
    if (j < N) {
        const int page = kv.block_table[(long long)p * kv.max_pages + j / kv.page_size];
        if (page >= 0 && page < kv.num_pages) c3 = page;
        else {
            if (status) atomicOr(status, MAGE_DEV_BAD_PAGE);
            return true;
        }
    }
    return false;
}

// Paged caches: the page-table entry of the 64-key box at logical position j (-2 beyond the prefix), and the box
// coordinates from an entry looked up earlier.  The producers look entries up a tile or two ahead of their use: a lookup
// is a dependent global load of about half a microsecond, and four of them per tile (two boxes each of K and V) on the
// producer's critical path would take longer than the tile's arithmetic.
__device__ __forceinline__ int page_entry(const KvView &kv, int p, int j, int N) {
    return j < N ? kv.block_table[(long long)p * kv.max_pages + j / kv.page_size] : -2;
}
__device__ __forceinline__ bool paged_box_coords(const KvView &kv, int h, int j, int entry, int &c1, int &c2, int &c3, unsigned *status) {
    c1 = j % kv.page_size;
    c2 = h;
    c3 = kv.num_pages;                     // out of range: zero fill
    if (entry == -2) return false;         // beyond the prefix
    if (entry >= 0 && entry < kv.num_pages) { c3 = entry; return false; }
    if (status) atomicOr(status, MAGE_DEV_BAD_PAGE);
    return true;
}

// ------------------------------------------------------------------------------------------------------------
// Block-score kernel (Eq. 4): score[j] = 1/M * sum_r exp2(scale_log2 * <q_r, k_j> - lse2_r).
// Orientation: keys are the MMA M dimension (TMEM lanes), query rows the N dimension (TMEM columns), so each
// thread owns one key and its sum over rows needs no cross-thread reduction.  One CTA walks `tiles_per_cta`
// consecutive 128-key tiles of one KV head.
// The kernel is bound by the special-function unit (128*M exponentials per tile at 16 per clock per SM, against
// 4*M clocks of MMA), so the layout's job is to keep that unit busy through the hand-offs.  A unit of work is
// (key tile, half of the query rows): S^T of a unit is 128 lanes x <=128 columns, TMEM holds four of them, and each
// of the four warpgroups owns one buffer: warpgroup w takes the units u = w (mod 4), i.e. tiles of parity w/2 and
// row half w%2.  While one warpgroup waits for the MMA to refill its buffer the other three are in their
// exponentials, so the hand-off latency is hidden without any warpgroup-to-warpgroup barrier.  The row-half-1
// warpgroup of a tile hands its 128 partial sums to the row-half-0 warpgroup through shared memory, which adds them
// (fixed order) one unit late and stores the score.
// ------------------------------------------------------------------------------------------------------------
// Optional tile list of the score pass (pruned selection): per (problem, KV head) an ascending list of key-tile numbers to
// score instead of all tiles.  count is per KV head, or per problem when count_per_problem is set; compact, when given,
// receives the listed tiles' scores in list order ([P*H_kv][stride][128]) and compact_lens[p] their number of entries.
struct ScoreTileList {
    const int *tiles = nullptr;
    const int *count = nullptr;
    int stride = 0, count_per_problem = 0;
    float *compact = nullptr;
    int *compact_lens = nullptr;
};

constexpr int kScoreStages = 4;
constexpr int kScoreWgs = 4;
constexpr int kScoreThreads = kScoreWgs * 128 + 64;
constexpr int kScoreProducerWarp = kScoreWgs * 4, kScoreMmaWarp = kScoreWgs * 4 + 1;
constexpr int kScoreQBytes = 2 * 256 * 128;           // up to 256 query rows, two d-halves
constexpr size_t kScoreSmemBytes = 1024 + kScoreQBytes + kScoreStages * kTileBytes + (256 + 2 * 128) * sizeof(float) + 320;

// K8: queries and keys arrive as e4m3 codes (rows of 128 bytes, one 128-byte swizzle atom per row, so a tile is one
// d-"half" of the 16-bit layout), the products run on the 8-bit MMA kind, and the head's factor s_q s_k (qk_scale) goes
// into the exponent's scale.  Everything after the logits is the same code.
template <bool K8>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, KvView kv, Plan plan,
             int row_begin, int rows, int tiles_per_cta, float scale_log2, const float *__restrict__ ws,
             float *__restrict__ scores, int accumulate, unsigned *status, ScoreTileList list, const float *__restrict__ qk_scale) {
    using namespace ptx;
    pdl_wait();
    pdl_launch_dependents();
    const int z = blockIdx.y, p = z / kv.H_kv, h = z % kv.H_kv;
    if (K8) scale_log2 *= qk_scale[z];
    const int N = seq_len_of(kv, p);
    // list mode (pruned selection): the CTA walks entries [tile0, tile0 + n_my) of this head's ascending list of tile numbers
    const int *my_list = list.tiles ? list.tiles + (size_t)z * list.stride : nullptr;
    const int tiles_total = my_list ? min(list.count[list.count_per_problem ? p : z], list.stride) : (N + kTile - 1) / kTile;
    const int tile0 = blockIdx.x * tiles_per_cta;
    if (my_list && blockIdx.x == 0 && h == 0 && threadIdx.x == 0 && list.compact_lens) list.compact_lens[p] = tiles_total * kTile;
    if (tile0 >= tiles_total) return;
    const int n_my = min(tiles_per_cta, tiles_total - tile0);
    auto tile_of = [&](int t) { return my_list ? my_list[tile0 + t] : tile0 + t; };     // actual key tile of the CTA's t-th

    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *q_s = base, *k_s = base + kScoreQBytes;
    float *neg_lse_s = reinterpret_cast<float *>(k_s + kScoreStages * kTileBytes);
    float *part_s = neg_lse_s + 256;                   // [2 tile parities][128] partial sums of the row-half-1 warpgroups
    uint64_t *bars = reinterpret_cast<uint64_t *>(part_s + 2 * 128);
    enum { Q_FULL = 0, FULL = 1, EMPTY = FULL + kScoreStages, T_FULL = EMPTY + kScoreStages, T_EMPTY = T_FULL + 4,
           P_FULL = T_EMPTY + 4, P_EMPTY = P_FULL + 2, N_BARS = P_EMPTY + 2 };
    uint32_t *tmem_ptr_s = reinterpret_cast<uint32_t *>(bars + N_BARS);
    volatile int *abort_s = reinterpret_cast<volatile int *>(tmem_ptr_s + 1);
    // per key tile (ring of 16, far deeper than the producer can run ahead): bit kh set = the 64-key box kh of the tile
    // came from a page id out of range; its keys get score 0
    volatile int *tile_bad_s = reinterpret_cast<volatile int *>(tmem_ptr_s + 3);
    auto bar = [&](int i) { return smem_u32(bars + i); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rows64 = (rows + 63) & ~63;
    // the two row halves: [0, rows_lo) and [rows_lo, rows); rows_lo is a multiple of 8 rows (one swizzle atom)
    // With at most 128 query rows (e.g. G = 4, B = 32) a unit is a whole tile instead: the four warpgroups take the tiles
    // i = 0, 1, 2, 3 (mod 4), each with all the rows, and nothing is exchanged between warpgroups ("quad" mode).  Half-row
    // units of 64 columns would spend as long in their hand-offs as in their exponentials.
    const bool quad = rows <= 128;
    const int rows_lo = quad ? rows : min(rows, (((rows + 1) >> 1) + 7) & ~7), rows_hi = rows - rows_lo;
    const int n_units = rows_hi > 0 ? 2 : 1;           // units per tile

    if (tid < 16) tile_bad_s[tid] = 0;
    if (tid == 0) {
        abort_s[0] = 0;
        abort_s[1] = 0;                                    // the ordinary wait limit
        mbar_init(bar(Q_FULL), 1);
        for (int s = 0; s < kScoreStages; ++s) { mbar_init(bar(FULL + s), 1); mbar_init(bar(EMPTY + s), 1); }
        for (int b = 0; b < 4; ++b) { mbar_init(bar(T_FULL + b), 1); mbar_init(bar(T_EMPTY + b), 4); }   // one arrival per warp
        for (int b = 0; b < 2; ++b) { mbar_init(bar(P_FULL + b), 4); mbar_init(bar(P_EMPTY + b), 4); }
        fence_mbar_init();
    }
    if (warp == kScoreMmaWarp) { tmem_alloc(smem_u32(tmem_ptr_s), 512); tmem_relinquish(); }
    if (tid < 256) neg_lse_s[tid] = tid < rows ? ws[plan.off_neg_lse + (size_t)z * plan.Mw + row_begin + tid] : 0.f;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_ptr_s;

    if (warp == kScoreProducerWarp) {
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            const int q_row0 = (p * kv.H_q + h * kv.G) * kv.B + row_begin;
            mbar_arrive_expect_tx(bar(Q_FULL), (K8 ? 1 : 2) * rows64 * 128);
            for (int dh = 0; dh < (K8 ? 1 : 2); ++dh)
                for (int rb = 0; rb < rows64 / 64; ++rb)
                    tma_load_2d(smem_u32(q_s + dh * (kScoreQBytes / 2) + rb * kBoxBytes), &map_q, bar(Q_FULL), dh * 64, q_row0 + rb * 64);
            const uint64_t pol_k = l2_policy_evict_first();       // last use of these K lines
            const bool paged = kv.page_size != 0;
            int pg_cur[2] = {-2, -2}, pg_nxt[2] = {-2, -2};        // page-table entries of the CTA's tile i and tile i + 1
            if (paged) {
                for (int kh = 0; kh < 2; ++kh) {
                    pg_cur[kh] = page_entry(kv, p, tile_of(0) * kTile + kh * 64, N);
                    pg_nxt[kh] = n_my > 1 ? page_entry(kv, p, tile_of(1) * kTile + kh * 64, N) : -2;
                }
            }
            int issued = 0;
            for (int i = 0; i < n_my; ++i) {
                const int slot = i % kScoreStages, u = i / kScoreStages;
                if (!mbar_wait(bar(EMPTY + slot), (u & 1) ^ 1, abort_s, status)) break;
                const int j0 = tile_of(i) * kTile;
                int c1[2], c2[2], c3[2], bad = 0;
                if (paged) {
                    for (int kh = 0; kh < 2; ++kh)
                        if (paged_box_coords(kv, h, j0 + kh * 64, pg_cur[kh], c1[kh], c2[kh], c3[kh], status)) bad |= 1 << kh;
                    tile_bad_s[i & 15] = bad;                         // ordered before the tile's FULL phase by the arrive below
                    for (int kh = 0; kh < 2; ++kh) {
                        pg_cur[kh] = pg_nxt[kh];
                        pg_nxt[kh] = i + 2 < n_my ? page_entry(kv, p, tile_of(i + 2) * kTile + kh * 64, N) : -2;
                    }
                } else {
                    for (int kh = 0; kh < 2; ++kh) cache_box_coords(kv, p, h, j0 + kh * 64, N, c1[kh], c2[kh], c3[kh], nullptr);
                }
                mbar_arrive_expect_tx(bar(FULL + slot), K8 ? kHalfBytes : kTileBytes);
                for (int kh = 0; kh < 2; ++kh)
                    for (int dh = 0; dh < (K8 ? 1 : 2); ++dh)
                        tma_load_4d_hint(smem_u32(k_s + slot * kTileBytes + dh * kHalfBytes + kh * kBoxBytes), &map_k, bar(FULL + slot), dh * 64, c1[kh], c2[kh], c3[kh], pol_k);
                issued = i + 1;
            }
            if (*abort_s) {   // give the copies already in flight a bounded chance to land before the CTA exits
                for (int i = max(0, issued - kScoreStages); i < issued; ++i) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(bar(FULL + i % kScoreStages), (i / kScoreStages) & 1) && clock64() - t0 < 2000000) {}
                }
            }
        }
    } else if (warp == kScoreMmaWarp) {
        if (lane == 0) {
            const uint32_t idesc_lo = K8 ? idesc_e4m3_f32((rows_lo + 15) & ~15) : idesc_bf16_f32((rows_lo + 15) & ~15, false, false);
            const uint32_t idesc_hi = K8 ? idesc_e4m3_f32(max(16, (rows_hi + 15) & ~15)) : idesc_bf16_f32(max(16, (rows_hi + 15) & ~15), false, false);
            bool ok = mbar_wait(bar(Q_FULL), 0, abort_s, status);
            for (int i = 0; ok && i < n_my; ++i) {
                const int slot = i % kScoreStages, su = i / kScoreStages;
                if (!mbar_wait(bar(FULL + slot), su & 1, abort_s, status)) break;
                const uint32_t k_addr = smem_u32(k_s + slot * kTileBytes), q_addr = smem_u32(q_s);
                for (int rh = 0; rh < n_units && ok; ++rh) {
                    const int buf = quad ? (i & 3) : (i & 1) * 2 + rh, use = quad ? i >> 2 : i >> 1;     // buffer = warpgroup that consumes it
                    if (!mbar_wait(bar(T_EMPTY + buf), (use & 1) ^ 1, abort_s, status)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (K8) {                                  // 32 one-byte elements of d per step: the whole row is one atom
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t a = smem_desc_sw128(k_addr + ks * 32, 16, 1024);
                            const uint64_t b = smem_desc_sw128(q_addr + ks * 32 + rh * rows_lo * 128, 16, 1024);
                            umma_ss_f8(tmem_base + buf * 128, a, b, rh ? idesc_hi : idesc_lo, ks > 0);
                        }
                    } else {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                            const uint64_t a = smem_desc_sw128(k_addr + off, 16, 1024);
                            const uint64_t b = smem_desc_sw128(q_addr + (ks >> 2) * (kScoreQBytes / 2) + (ks & 3) * 32 + rh * rows_lo * 128, 16, 1024);
                            umma_ss(tmem_base + buf * 128, a, b, rh ? idesc_hi : idesc_lo, ks > 0);
                        }
                    }
                    umma_commit(bar(T_FULL + buf));
                }
                umma_commit(bar(EMPTY + slot));
            }
        }
    } else {
        const int wg = warp >> 2, w4 = warp & 3, key = w4 * 32 + lane;
        const int par = quad ? wg : wg >> 1, rh = quad ? 0 : wg & 1;      // tiles i = par (mod step) and row half of this warpgroup
        const int step = quad ? 4 : 2;
        const float inv_m = 1.f / (float)kv.M;
        float *srow = scores + (size_t)z * kv.N_max;
        const int col_lo = rh ? rows_lo : 0, n_cols = rh ? rows_hi : rows_lo;      // my columns: neg_lse index = col_lo + c
        const uint64_t c2 = pack2(scale_log2, scale_log2);
        const uint32_t taddr = tmem_base + wg * 128 + ((uint32_t)(w4 * 32) << 16);
        float prev_sum = 0.f;
        int prev_tile = -1;
        bool prev_bad = false;
        // row half 0: add the other half's partial sum of tile t to its own and store the score (0 for a key whose page
        // id was out of range: it is skipped by the attention pass, so it carries no probability)
        auto finish = [&](int t, float own, bool bad) -> bool {
            float v = own;
            if (n_units == 2) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar(P_FULL + par), (t >> 1) & 1, abort_s, status))) return false;
                v += part_s[par * 128 + key];
                mbar_arrive_warp(bar(P_EMPTY + par));
            }
            v = bad ? 0.f : v * inv_m;
            const int j = tile_of(t) * kTile + key;
            if (j < N) srow[j] = accumulate ? srow[j] + v : v;
            if (list.compact) {                                  // the same scores in list order, zeros past the prefix
                float *c = list.compact + ((size_t)z * list.stride + tile0 + t) * kTile + key;
                *c = j < N ? (accumulate ? *c + v : v) : 0.f;
            }
            return true;
        };
        bool ok = true;
        if (n_cols > 0) {
            for (int i = par; i < n_my; i += step) {
                const int use = quad ? i >> 2 : i >> 1;
                if (!__all_sync(0xffffffffu, mbar_wait(bar(T_FULL + wg), use & 1, abort_s, status))) { ok = false; break; }
                tc_fence_after_sync();
                const bool key_bad = (tile_bad_s[i & 15] >> (key >> 6)) & 1;
                float tail = 0.f;
                uint64_t acc_a = pack2(0.f, 0.f), acc_b = acc_a;
                // one step = 8 columns = 4 pairs; the TMEM load of the next step is in flight while this one is processed
                auto step = [&](const uint32_t (&r)[8], int c0) {
                    if (c0 + 8 <= n_cols) {
                        const float4 *nl4 = reinterpret_cast<const float4 *>(neg_lse_s + col_lo + c0);
                        const float4 n0 = nl4[0], n1 = nl4[1];
                        uint64_t x[4];
                        x[0] = fma2(pack2(__uint_as_float(r[0]), __uint_as_float(r[1])), c2, pack2(n0.x, n0.y));
                        x[1] = fma2(pack2(__uint_as_float(r[2]), __uint_as_float(r[3])), c2, pack2(n0.z, n0.w));
                        x[2] = fma2(pack2(__uint_as_float(r[4]), __uint_as_float(r[5])), c2, pack2(n1.x, n1.y));
                        x[3] = fma2(pack2(__uint_as_float(r[6]), __uint_as_float(r[7])), c2, pack2(n1.z, n1.w));
                        ex2_mufu2_n(x);
                        acc_a = add2(acc_a, x[0]); acc_b = add2(acc_b, x[1]);
                        acc_a = add2(acc_a, x[2]); acc_b = add2(acc_b, x[3]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (c0 + e < n_cols) tail += ex2(fmaf(__uint_as_float(r[e]), scale_log2, neg_lse_s[col_lo + c0 + e]));
                    }
                };
                // The usual column counts (128, 64, and 112 = half of G*B = 224) run fully unrolled, 16 columns per step:
                // no loop counters, compares or branches, constant offsets, half as many TMEM loads and waits.  The
                // warps of this kernel issue more than half of all cycles, so instructions saved here are time saved.
                auto step16 = [&](const uint32_t (&r)[16], int c0) {
                    const float4 *nl4 = reinterpret_cast<const float4 *>(neg_lse_s + col_lo + c0);
                    uint64_t x[8];
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const float4 nq = nl4[q4];
                        x[2 * q4] = fma2(pack2(__uint_as_float(r[4 * q4]), __uint_as_float(r[4 * q4 + 1])), c2, pack2(nq.x, nq.y));
                        x[2 * q4 + 1] = fma2(pack2(__uint_as_float(r[4 * q4 + 2]), __uint_as_float(r[4 * q4 + 3])), c2, pack2(nq.z, nq.w));
                    }
                    ex2_mufu2_n(x);
#pragma unroll
                    for (int q = 0; q < 8; q += 2) { acc_a = add2(acc_a, x[q]); acc_b = add2(acc_b, x[q + 1]); }
                };
                auto sweep16 = [&](auto n_steps_tag) {
                    constexpr int kSteps = decltype(n_steps_tag)::value;
                    uint32_t ua[16], ub[16];
                    tmem_ld16(taddr, ua);
#pragma unroll
                    for (int st = 0; st < kSteps; st += 2) {
                        tmem_wait_ld(ua);
                        if (st + 1 < kSteps) tmem_ld16(taddr + (st + 1) * 16, ub);
                        step16(ua, st * 16);
                        if (st + 1 < kSteps) {
                            tmem_wait_ld(ub);
                            if (st + 2 < kSteps) tmem_ld16(taddr + (st + 2) * 16, ua);
                            step16(ub, (st + 1) * 16);
                        }
                    }
                };
                if (n_cols == 128) {
                    sweep16(std::integral_constant<int, 8>{});
                } else if (n_cols == 112) {
                    sweep16(std::integral_constant<int, 7>{});
                } else if (n_cols == 64) {
                    sweep16(std::integral_constant<int, 4>{});
                } else {
                    uint32_t ra[8], rb[8];
                    tmem_ld8(taddr, ra);
                    for (int c0 = 0; c0 < n_cols; c0 += 16) {
                        tmem_wait_ld(ra);
                        if (c0 + 8 < n_cols) tmem_ld8(taddr + c0 + 8, rb);
                        step(ra, c0);
                        if (c0 + 8 < n_cols) {
                            tmem_wait_ld(rb);
                            if (c0 + 16 < n_cols) tmem_ld8(taddr + c0 + 16, ra);
                            step(rb, c0 + 8);
                        }
                    }
                }
                tc_fence_before_sync();
                mbar_arrive_warp(bar(T_EMPTY + wg));
                float a0, a1, b0, b1;
                unpack2(acc_a, a0, a1); unpack2(acc_b, b0, b1);
                const float sum = ((a0 + a1) + (b0 + b1)) + tail;
                if (rh == 1) {
                    if (!__all_sync(0xffffffffu, mbar_wait(bar(P_EMPTY + par), (use & 1) ^ 1, abort_s, status))) { ok = false; break; }
                    part_s[par * 128 + key] = sum;
                    mbar_arrive_warp(bar(P_FULL + par));
                } else {
                    // finish the previous tile of this parity now, one unit late, so this warpgroup never waits for its partner
                    if (prev_tile >= 0 && !finish(prev_tile, prev_sum, prev_bad)) { ok = false; break; }
                    prev_sum = sum;
                    prev_tile = i;
                    prev_bad = key_bad;
                }
            }
            if (ok && rh == 0 && prev_tile >= 0) finish(prev_tile, prev_sum, prev_bad);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kScoreMmaWarp) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

// ------------------------------------------------------------------------------------------------------------
// Attention kernel (Algorithm 1: "Attn(Q, K, V, C)" over one chunk of the prefix, and "SparseAttn" over the
// selected rows): flash-style online softmax with both contractions on tcgen05.
//
// One CTA owns up to 256 query rows of one KV head (two 128-row M-tiles, one per softmax warpgroup) and walks
// 128-key tiles.  Per tile and M-tile:  S = Q K^T  (SS MMA into TMEM, 128 fp32 columns)  ->  the warpgroup
// reads its rows of S, keeps a running reference maximum and sum per row, writes P = exp2(.) as bf16 over the
// first 64 columns of S  ->  O += P V  (A operand = P from TMEM, B operand = the V tile in its natural
// [key][d] layout, i.e. MN-major).  While one warpgroup is in its softmax the tensor pipe works for the other.
// O stays in TMEM for the whole chunk.  A row rescales its O only when its maximum grew by more than 2^8;
// that happens between "S(i) complete" and "P(i) ready", when no MMA touches O of that M-tile: tcgen05.commit
// tracks every MMA issued before it, and PV(i-1) is issued before QK(i).
//
// DENSE  (SPARSE = false): K/V tiles arrive by TMA from the cache (or from the block's own keys for the last
//         chunk index); the result is the unnormalised partial (O, m, l) of the chunk, merged by combine_kernel.
// SPARSE (SPARSE = true): four producer warps gather the k_eff selected cache rows (then the block's keys) into the
//         same swizzled layout -- one row per thread as two 64 x 1 TMA boxes when the cache has a single row pitch,
//         16-byte cp.async otherwise; the result is the final bf16 output (or a partial one per CTA when a head's
//         keys are split over several CTAs).
// With a single M-tile (G*B <= 128) the two warpgroups take alternate key tiles of the same rows instead.
// ------------------------------------------------------------------------------------------------------------
constexpr int kAttnSlotsDense = 5;                     // ring of K/V tile slots: K(0) V(0) K(1) V(1) ...
constexpr int kAttnSlotsSparse = 4;                    // one slot less: the room holds the gathered rows' offset table
constexpr int kSparseTableCap = 4096;                  // selected rows whose cache offsets are tabulated in shared memory
constexpr int kAttnQBytes = 2 * kTileBytes;            // two M-tiles of 128 rows
constexpr size_t kAttnSmemBytesDense = 1024 + kAttnQBytes + kAttnSlotsDense * kTileBytes + 512;
constexpr size_t kAttnSmemBytesSparse = 1024 + kAttnQBytes + kAttnSlotsSparse * kTileBytes + 512 + kSparseTableCap * sizeof(int);
constexpr float kRescaleThreshold = 8.f;               // log2 units
// Reuse step: warps that issue the row gathers.  A TMA request keeps the issuing warp for about 115 cycles whatever it
// fetches, and the lanes of a warp issue one after the other, so the gather rate of a CTA is set by the number of warps
// that issue: seven fill a 512-thread CTA beside the eight softmax warps and the MMA warp.
constexpr int kSparseProducerWarps = 7;
constexpr int kSparseThreads = 256 + kSparseProducerWarps * 32 + 32;

// Reuse step, error path only: bits of the 32 selected keys from list position t0 on that must be left out of the softmax
// (index outside the prefix, or its page id out of range).  row_tab: the CTA's table of resolved rows (-1 = left out), or
// null when the budget exceeds the table; then idx (this head's index list, already shifted to the CTA's first key) and
// the problem's row of the page table are consulted.  Kept out of line: the hot loops must not pay registers for it.
__device__ __noinline__ uint32_t sparse_bad_cols(const int *row_tab, const int *idx, int t0, int n_cache, int N,
                                                 const int *table_row, int page_size, int num_pages) {
    uint32_t badm = 0;
    for (int e = 0; e < 32 && t0 + e < n_cache; ++e) {
        bool b;
        if (row_tab) {
            b = row_tab[t0 + e] < 0;
        } else {
            const int j = idx[t0 + e];
            b = j < 0 || j >= N;
            if (!b && page_size) {
                const int pg = table_row[j / page_size];
                b = pg < 0 || pg >= num_pages;
            }
        }
        if (b) badm |= 1u << e;
    }
    return badm;
}

// gather_rows > 0 (reuse step only): k, v, kb, vb are flat row lists (pitch gather_pitch elements) with 64 x 1 boxes.
// lse_only (exact pass only): the select stream's own pass -- row maxima and sums over the prefix, no V, no P V, no O.
struct AttnMaps {
    CUtensorMap q, k, v, kb, vb;
    int gather_rows = 0, gather_blk_rows = 0, gather_pitch = 0, lse_only = 0;
    // exact pass only, optional: per (KV head, 128-key tile, query row) the tile's unnormalised row sum and the reference it
    // was taken against, [P*H_kv][rowsum_tiles][Mw] pairs; sum * 2^(reference - row's log2-sum-exp) is the row's probability
    // mass on that tile, which the pruned selection adds up over rows into an upper bound for every key of the tile
    float2 *rowsum = nullptr;
    int rowsum_tiles = 0;
    int test_stall = 0;          // MAGE_FLAG_TEST_STALL: the exact pass never requests its first key tile and waits with the short limit
    const float *qk_scale = nullptr;   // 8-bit keys: s_q s_k per (problem, KV head); q, k, kb are then maps of e4m3 codes
    // 8-bit keys, reuse step with at most 256 query rows per KV head: the kernel codes the queries and the block's keys
    // itself (no kernel in front of it, no q / kb maps): the bf16 queries, and the key scale of each (problem, KV head)
    const __nv_bfloat16 *q_raw = nullptr;
    const float *k_scale = nullptr;
    // query rows per CTA (blockIdx.y counts groups of this many rows of a KV head): 256, or 128 for a reuse step that is split
    // over CTAs anyway -- a 128-row CTA writes half the partial result, which is most of what such a CTA spends its time on
    int rg_rows = 256;
};

// K8: queries and keys (cache and block) are e4m3 codes in rows of 128 bytes; a Q or K tile then fills the first d-"half"
// of its 32 KB region, Q K^T runs on the 8-bit MMA kind in four steps of 32 elements, and the head's s_q s_k goes into the
// softmax scale.  Values, P and P V are as in the 16-bit kernel.
template <bool SPARSE, bool K8 = false>
__global__ void __launch_bounds__(SPARSE ? kSparseThreads : 320, 1)
attn_kernel(const __grid_constant__ AttnMaps maps, KvView kv, Plan plan, const __nv_bfloat16 *__restrict__ k_blk,
            const __nv_bfloat16 *__restrict__ v_blk, const int *__restrict__ indices, const int *__restrict__ k_eff_arr, int k,
            float scale_log2, float *__restrict__ ws, __nv_bfloat16 *__restrict__ out, unsigned *status) {
    using namespace ptx;
    if (threadIdx.x == 0) MAGE_STAMP(0);
    MAGE_CLK(126);
    if (threadIdx.x < 5) prefetch_tensormap(&maps.q + threadIdx.x);    // (kernel parameters: no need to wait for the predecessor)
    pdl_wait();                      // everything below may read what the previous kernel in the stream wrote
    pdl_launch_dependents();
    if (threadIdx.x == 0) MAGE_STAMP(1);
    constexpr int kMmaWarp = SPARSE ? 8 + kSparseProducerWarps : 9;
    constexpr int kAttnSlots = SPARSE ? kAttnSlotsSparse : kAttnSlotsDense;
    const int chunk = blockIdx.x, rg = blockIdx.y, z = blockIdx.z, p = z / kv.H_kv, h = z % kv.H_kv;
    const int N = seq_len_of(kv, p);
    const bool fused_codes = K8 && SPARSE && maps.q_raw != nullptr;
    if (K8 && !fused_codes) scale_log2 *= maps.qk_scale[z];
    int n_keys, n_cache, j_begin = 0, first_idx = 0;
    bool blk_chunk = false;
    if (!SPARSE) {
        if (chunk < plan.n_chunks) {
            j_begin = chunk * plan.chunk_len;
            if (j_begin >= N) return;
            n_keys = n_cache = min(plan.chunk_len, N - j_begin);
        } else {
            blk_chunk = true;
            n_keys = kv.B;
            n_cache = 0;
        }
    } else {
        // (the thread's first selected index starts its way in before the problem's k_eff is read, so that the two cold
        // loads overlap; the unsplit launch only, where the CTA's list starts at the head's first index)
        if (gridDim.x == 1 && (int)threadIdx.x < k) first_idx = indices[(long long)z * k + threadIdx.x];
        n_cache = min(max(k_eff_arr[p], 0), k);
        n_keys = n_cache + kv.B;
    }
    // SPARSE with gridDim.x > 1: this CTA takes tiles [tile_lo, tile_lo + n_tiles) of the head's key list and writes
    // a partial result; key_off shifts the positions in that list.
    int key_off = 0, blk_shift = n_cache;     // block key number = local position - blk_shift
    if (SPARSE && gridDim.x > 1) {
        const int tiles_all = (n_keys + kTile - 1) / kTile, per = (tiles_all + gridDim.x - 1) / gridDim.x;
        const int tile_lo = chunk * per;
        if (tile_lo >= tiles_all) return;
        key_off = tile_lo * kTile;
        n_keys = min(n_keys - key_off, per * kTile);
        blk_shift = n_cache - key_off;
        n_cache = max(0, blk_shift);
    }
    const int n_tiles = (n_keys + kTile - 1) / kTile;
    // Reuse step: the last tile of the list usually holds little more than the block's own keys; it is gathered, multiplied
    // and exponentiated at its own width (a multiple of 16 keys) instead of a full 128.
    const int last_cols = SPARSE ? ((n_keys - (n_tiles - 1) * kTile + 15) & ~15) : kTile;
    const int rgr = SPARSE ? maps.rg_rows : 256;         // query rows per row group
    const int rows_here = min(rgr, kv.M - rg * rgr), n_mt = rows_here > 128 ? 2 : 1;
    // With a single M-tile the second softmax warpgroup and the second S/O regions would idle.  They take the
    // odd key tiles instead ("tile-parity mode"): two independent online-softmax pipelines over the same 128 rows,
    // each with its own reference, sum and O accumulator, merged by warpgroup 0 at the end.
    const bool tp = n_mt == 1;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *q_s = base, *kv_s = base + kAttnQBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(kv_s + kAttnSlots * kTileBytes);
    enum { Q_FULL = 0, FULL = 1, EMPTY = FULL + kAttnSlots, S_FULL = EMPTY + kAttnSlots, P_HALF = S_FULL + 2, P_FULL = P_HALF + 2,
           PVH_DONE = P_FULL + 2, O_DONE = PVH_DONE + 2, PUB = O_DONE + 1, N_BARS = PUB + 1 };
    uint32_t *tmem_ptr_s = reinterpret_cast<uint32_t *>(bars + N_BARS);
    volatile int *abort_s = reinterpret_cast<volatile int *>(tmem_ptr_s + 1);
    // Keys that must be left out of the softmax although their rows arrive as zeros.  SPARSE: `any_bad` below, one flag for
    // the CTA, set when any selected index or its page is out of range (every tile then takes the careful path and looks
    // its columns up).  DENSE: per key tile (ring of 8), bit kh set = the 64-key box kh of the tile came from a page id out
    // of range.
    volatile int *tile_bad_s = reinterpret_cast<volatile int *>(tmem_ptr_s + 4);
    int *row_tab = reinterpret_cast<int *>(tmem_ptr_s + 12);    // SPARSE: cache offset / 8 of each selected row, -1 = skip
    auto bar = [&](int i) { return smem_u32(bars + i); };
    auto slot_of = [](int L) { return L % kAttnSlots; };
    auto par_of = [](int L) { return (L / kAttnSlots) & 1; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < 8) tile_bad_s[tid] = 0;
    if (tid == 0) {
        abort_s[0] = 0;
        abort_s[1] = maps.test_stall;                        // non-zero: waits give up after ~1 ms instead of ~0.25 s
        mbar_init(bar(Q_FULL), 1);
        for (int s = 0; s < kAttnSlots; ++s) { mbar_init(bar(FULL + s), SPARSE ? (maps.gather_rows > 0 ? kSparseProducerWarps : 4) : 1); mbar_init(bar(EMPTY + s), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(S_FULL + b), 1);
            mbar_init(bar(P_HALF + b), 4);                  // one arrival per warp
            mbar_init(bar(P_FULL + b), 4);
            mbar_init(bar(PVH_DONE + b), 1);
        }
        mbar_init(bar(O_DONE), 1);
        mbar_init(bar(PUB), 4);
        fence_mbar_init();
        fence_proxy_async();
        // the queries start their way in at once: (d, row within the KV head's G*B rows, head); rows past the head read as zeros
        if (!fused_codes) {
            mbar_arrive_expect_tx(bar(Q_FULL), n_mt * (K8 ? kHalfBytes : kTileBytes));
            for (int mt = 0; mt < n_mt; ++mt)
                for (int dh = 0; dh < (K8 ? 1 : 2); ++dh)
                    for (int rb = 0; rb < 2; ++rb)
                        tma_load_3d(smem_u32(q_s + mt * kTileBytes + dh * kHalfBytes + rb * kBoxBytes), &maps.q, bar(Q_FULL), dh * 64,
                                    rg * rgr + mt * kTile + rb * 64, z);
        }
    }
    // 8-bit keys, coded here: every thread fetches its share of the head's bf16 queries (all G*B <= 256 rows: one row group)
    // and of the block's keys now, so that the loads run under the set-up and the index look-ups below.
    uint4 fq[8], fb[2];
    uint8_t *kb_stage = q_s + kHalfBytes;                 // [B][128] codes of the block's keys (the Q tile of M-tile 0 ends at 16 KB)
    if (K8 && SPARSE && fused_codes) {
        const uint4 *qv = reinterpret_cast<const uint4 *>(maps.q_raw + ((size_t)(p * kv.H_q + h * kv.G) * kv.B) * kD);
        const int n_q16 = kv.M * 8;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = tid + u * (int)blockDim.x;
            const bool in = j < n_q16;
            fq[2 * u] = in ? qv[2 * j] : make_uint4(0, 0, 0, 0);
            fq[2 * u + 1] = in ? qv[2 * j + 1] : make_uint4(0, 0, 0, 0);
        }
        const uint4 *bv = reinterpret_cast<const uint4 *>(k_blk + (size_t)z * kv.B * kD);
        const bool in = tid < kv.B * 8;
        fb[0] = in ? bv[2 * tid] : make_uint4(0, 0, 0, 0);
        fb[1] = in ? bv[2 * tid + 1] : make_uint4(0, 0, 0, 0);
    }
    if (warp == kMmaWarp) { tmem_alloc(smem_u32(tmem_ptr_s), 512); tmem_relinquish(); }
    // SPARSE: resolve every selected index to a cache row once (shared by the K and V gathers): bounds check,
    // page-table lookup, offset in 16-byte units.  Budgets beyond the table are resolved on the fly.
    auto resolve_idx = [&](int j) -> int {
        if (j < 0 || j >= N) {
            if (status) atomicOr(status, MAGE_DEV_BAD_INDEX);
            return -1;
        }
        const long long off = cache_row_offset(kv, p, h, j, status);
        if (off < 0) return -1;
        return maps.gather_rows > 0 ? (int)(off / maps.gather_pitch) : (int)(off >> 3);
    };
    auto resolve = [&](int t) -> int { return resolve_idx(indices[(long long)z * k + key_off + t]); };
    const bool use_tab = SPARSE && n_cache <= kSparseTableCap;
    int my_bad = 0;
    if (SPARSE) {
        for (int t = tid; t < n_cache; t += blockDim.x) {
            const int o = gridDim.x == 1 && t == tid ? resolve_idx(first_idx) : resolve(t);
            if (use_tab) row_tab[t] = o;
            if (o < 0) my_bad = 1;
        }
    }
    if (K8 && SPARSE && fused_codes) {
        // s_q = amax / 448 over the head's query rows, as the kernel in front of the other 8-bit calls takes it: the same
        // numbers in the same arithmetic, so the codes are the same bytes
        float *red = reinterpret_cast<float *>(kb_stage + 64 * 128);
        float m = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) m = k8::amax8(fq[u], m);
#pragma unroll
        for (int w = 16; w; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
        if (lane == 0) red[warp] = m;
        __syncthreads();
        m = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, red[w]);
        const float s_q = k8::scale_of(m), s_k = maps.k_scale[z];
        scale_log2 *= s_q * s_k;
        // Q codes into the 128-byte-swizzled tile (row r of M-tile mt at r * 128, 16-byte piece c at (c ^ (r & 7)) * 16); rows
        // beyond the head's last query row are zero, as the tensor map's fill would leave them
        const int n_q16 = kv.M * 8, n_all = n_mt * kTile * 8;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = tid + u * (int)blockDim.x;
            if (j < n_all) {
                const int R = j >> 3, c = j & 7, mt_ = R >> 7, r = R & 127;
                const uint4 code = j < n_q16 ? k8::code16(fq[2 * u], fq[2 * u + 1], s_q) : make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4 *>(q_s + mt_ * kTileBytes + r * 128 + ((c ^ (r & 7)) << 4)) = code;
            }
        }
        if (tid < kv.B * 8) *reinterpret_cast<uint4 *>(kb_stage + tid * 16) = k8::code16(fb[0], fb[1], s_k);
        fence_proxy_async();                               // the tensor pipe reads the Q tile through the async proxy
    }
    tc_fence_before_sync();
    const int any_bad = __syncthreads_or(my_bad);
    tc_fence_after_sync();
    if (K8 && SPARSE && fused_codes && tid == 0) mbar_arrive(bar(Q_FULL));     // the Q tile is in place (no copy to wait for)
    if (threadIdx.x == 0) MAGE_STAMP(2);
    const uint32_t tmem_base = *tmem_ptr_s;

    if (warp >= 8 && warp != kMmaWarp) {
        // ------------------------------------------------------------------ producers
        if (!SPARSE) {
            if (lane == 0) {
                const int blk_rows_total = kv.P * kv.H_kv * kv.B;
                // The score pass reads K again right after this pass and its merge: K lines are marked to stay in L2, V lines
                // (read once) to leave first.  Whether K survives depends on how much of it the launch covers (one layer
                // of a 32K prefix: 32 MB, it does; a 28-layer 128K batch streams 3.8 GB of K, it does not).
                const uint64_t pol_k = l2_policy_evict_last(), pol_v = l2_policy_evict_first();
                int issued = 0;
                if (kv.page_size != 0 && !blk_chunk) {
                    // paged cache: page-table entries of tile i and tile i + 1 are held in registers, looked up a tile ahead
                    int pg_cur[2], pg_nxt[2];
                    for (int kh = 0; kh < 2; ++kh) {
                        pg_cur[kh] = page_entry(kv, p, j_begin + kh * 64, N);
                        pg_nxt[kh] = page_entry(kv, p, j_begin + kTile + kh * 64, N);
                    }
                    for (int L = 0; L < 2 * n_tiles; ++L) {
                        const int i = L >> 1, is_v = L & 1, slot = slot_of(L);
                        if (!mbar_wait(bar(EMPTY + slot), par_of(L) ^ 1, abort_s, status)) break;
                        if (maps.test_stall) break;            // test hook: K(0) is never requested, so nothing is in flight
                        if (maps.lse_only && is_v) {           // no values in this mode: the slot's phase is completed empty-handed
                            mbar_arrive(bar(FULL + slot));
                        } else {
                            int c1[2], c2[2], c3[2], bad = 0;
                            for (int kh = 0; kh < 2; ++kh)
                                if (paged_box_coords(kv, h, j_begin + i * kTile + kh * 64, pg_cur[kh], c1[kh], c2[kh], c3[kh], is_v ? nullptr : status)) bad |= 1 << kh;
                            if (!is_v) tile_bad_s[i & 7] = bad;     // ordered before K(i)'s FULL phase by the arrive below
                            const int n_dh = K8 && !is_v ? 1 : 2;
                            mbar_arrive_expect_tx(bar(FULL + slot), n_dh * kHalfBytes);
                            const uint32_t dst = smem_u32(kv_s + slot * kTileBytes);
                            for (int kh = 0; kh < 2; ++kh)
                                for (int dh = 0; dh < n_dh; ++dh)
                                    tma_load_4d_hint(dst + dh * kHalfBytes + kh * kBoxBytes, is_v ? &maps.v : &maps.k, bar(FULL + slot), dh * 64, c1[kh], c2[kh], c3[kh], is_v ? pol_v : pol_k);
                        }
                        if (is_v) {                            // tile i + 1 becomes current, tile i + 2 is looked up
                            for (int kh = 0; kh < 2; ++kh) {
                                pg_cur[kh] = pg_nxt[kh];
                                pg_nxt[kh] = page_entry(kv, p, j_begin + (i + 2) * kTile + kh * 64, N);
                            }
                        }
                        issued = L + 1;
                    }
                } else {
                    for (int L = 0; L < 2 * n_tiles; ++L) {
                        const int i = L >> 1, is_v = L & 1, slot = slot_of(L);
                        if (!mbar_wait(bar(EMPTY + slot), par_of(L) ^ 1, abort_s, status)) break;
                        if (maps.test_stall) break;            // test hook: K(0) is never requested, so nothing is in flight
                        if (maps.lse_only && is_v) {           // no values in this mode: the slot's phase is completed empty-handed
                            mbar_arrive(bar(FULL + slot));
                            issued = L + 1;
                            continue;
                        }
                        const int n_dh = K8 && !is_v ? 1 : 2;
                        mbar_arrive_expect_tx(bar(FULL + slot), n_dh * kHalfBytes);
                        const uint32_t dst = smem_u32(kv_s + slot * kTileBytes);
                        for (int kh = 0; kh < 2; ++kh) {
                            if (!blk_chunk) {
                                int c1, c2, c3;
                                cache_box_coords(kv, p, h, j_begin + i * kTile + kh * 64, N, c1, c2, c3, nullptr);
                                for (int dh = 0; dh < n_dh; ++dh)
                                    tma_load_4d_hint(dst + dh * kHalfBytes + kh * kBoxBytes, is_v ? &maps.v : &maps.k, bar(FULL + slot), dh * 64, c1, c2, c3, is_v ? pol_v : pol_k);
                            } else {
                                const int row = (i == 0 && kh == 0) ? z * kv.B : blk_rows_total + 64;   // beyond the tensor: zero fill
                                for (int dh = 0; dh < n_dh; ++dh)
                                    tma_load_2d(dst + dh * kHalfBytes + kh * kBoxBytes, is_v ? &maps.vb : &maps.kb, bar(FULL + slot), dh * 64, row);
                            }
                        }
                        issued = L + 1;
                    }
                }
                if (*abort_s) {
                    for (int L = max(0, issued - kAttnSlots); L < issued; ++L) {
                        const long long t0 = clock64();
                        while (!mbar_try_wait(bar(FULL + slot_of(L)), par_of(L)) && clock64() - t0 < 2000000) {}
                    }
                }
            }
        } else {
            const int pt = tid - 256, cchunk = pt & 15, r0 = pt >> 4;
            if (maps.gather_rows > 0) {
                // TMA row gather, four rows per request: the cache is one 2-D tensor of 256-byte rows with a 64 x 1 box, and a
                // request names a column (d-half) and four row numbers, whose 128-byte halves land in four consecutive
                // rows of the swizzled tile.  Rows that do not exist (a bad index, the tail of the last tile) are named
                // beyond the tensor and arrive as zeros.
                int issued = 0;
                for (int L = 0; L < 2 * n_tiles; ++L) {
                    const int i = L >> 1, is_v = L & 1, slot = slot_of(L);
                    if (!__all_sync(0xffffffffu, mbar_wait(bar(EMPTY + slot), par_of(L) ^ 1, abort_s, status))) break;
                    // rows of this tile that are used at all (a multiple of 16), and this warp's share of them
                    // Requests of a tile: (group of four consecutive list positions, d-half), 64 for a full tile, fewer for
                    // the last one; request o goes to warp o % 7, lane o / 7.  Each warp announces its share of the bytes.
                    const int pw = pt >> 5;
                    // (8-bit keys: a key row is one 128-byte piece, so a K tile takes half as many requests)
                    const bool one_piece = K8 && !is_v;
                    const int n_req = ((i == n_tiles - 1 ? last_cols : kTile) >> 2) * (one_piece ? 1 : 2);
                    const int mine = n_req > pw ? (n_req - pw + kSparseProducerWarps - 1) / kSparseProducerWarps : 0;
                    if (K8 && fused_codes && !is_v) {
                        // Keys coded in this kernel: cache rows come by TMA as above; the block's rows are copied from the staged
                        // codes with plain stores (swizzled by hand), rows past the list are zero.  A lane first writes what it
                        // copies itself and makes it visible to the tensor pipe, then the warp announces exactly the bytes its TMA
                        // requests will bring, then those are issued.
                        const int o = lane * kSparseProducerWarps + pw, r_in_tile = o * 4, t0 = i * kTile + r_in_tile;
                        const int n_c = lane < mine ? min(4, max(0, n_cache - t0)) : 0;     // rows of the group that are cache rows
                        uint8_t *dst_g = kv_s + slot * kTileBytes + r_in_tile * 128;
                        int rows[4];
                        if (lane < mine) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int t = t0 + e, r = r_in_tile + e;
                                if (e < n_c) {
                                    const int ro = use_tab ? row_tab[t] : resolve(t);
                                    rows[e] = ro >= 0 ? ro : maps.gather_rows;          // beyond the tensor: zero fill
                                } else {
                                    const uint4 *src = reinterpret_cast<const uint4 *>(kb_stage + (t - blk_shift) * 128);
#pragma unroll
                                    for (int c = 0; c < 8; ++c)
                                        *reinterpret_cast<uint4 *>(dst_g + e * 128 + ((c ^ (r & 7)) << 4)) = t < n_keys ? src[c] : make_uint4(0, 0, 0, 0);
                                }
                            }
                            if (n_c < 4) fence_proxy_async();
                        }
                        const int tx = __reduce_add_sync(0xffffffffu, n_c * 128);
                        __syncwarp();                          // the lanes' stores and fences come before the warp's arrival
                        if (lane == 0) {
                            if (tx > 0) mbar_arrive_expect_tx(bar(FULL + slot), tx);
                            else mbar_arrive(bar(FULL + slot));
                        }
                        __syncwarp();
                        if (n_c == 4) {
                            tma_gather4_2d(smem_u32(dst_g), &maps.k, bar(FULL + slot), 0, rows[0], rows[1], rows[2], rows[3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (e < n_c) tma_load_2d(smem_u32(dst_g + e * 128), &maps.k, bar(FULL + slot), 0, rows[e]);
                        }
                        if (tid == 256) MAGE_STAMP(40 + L);
                        issued = L + 1;
                        continue;
                    }
                    if (lane == 0) {
                        if (mine > 0) mbar_arrive_expect_tx(bar(FULL + slot), mine * 512);
                        else mbar_arrive(bar(FULL + slot));
                    }
                    __syncwarp();
                    if (lane < mine) {
                        const int o = lane * kSparseProducerWarps + pw;
                        const int r_in_tile = (one_piece ? o : o >> 1) * 4, dh = one_piece ? 0 : o & 1, t0 = i * kTile + r_in_tile;
                        int rows[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int t = t0 + e;
                            if (t < n_cache) {
                                const int ro = use_tab ? row_tab[t] : resolve(t);
                                rows[e] = ro >= 0 ? ro : maps.gather_rows;          // beyond the tensor: zero fill
                            } else {
                                rows[e] = t < n_keys ? z * kv.B + (t - blk_shift) : maps.gather_blk_rows;
                            }
                        }
                        const uint32_t dst = smem_u32(kv_s + slot * kTileBytes + dh * kHalfBytes + r_in_tile * 128);
                        if (t0 + 3 < n_cache) {
                            tma_gather4_2d(dst, is_v ? &maps.v : &maps.k, bar(FULL + slot), dh * 64, rows[0], rows[1], rows[2], rows[3]);
                        } else if (t0 >= n_cache) {
                            tma_gather4_2d(dst, is_v ? &maps.vb : &maps.kb, bar(FULL + slot), dh * 64, rows[0], rows[1], rows[2], rows[3]);
                        } else {                                                    // the group straddles the end of the selected rows
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                tma_load_2d(dst + e * 128, t0 + e < n_cache ? (is_v ? &maps.v : &maps.k) : (is_v ? &maps.vb : &maps.kb), bar(FULL + slot), dh * 64, rows[e]);
                        }
                    }
                    if (tid == 256) MAGE_STAMP(40 + L);
                    issued = L + 1;
                }
                if (*abort_s) {                                        // let the copies in flight land before the CTA leaves
                    for (int L = max(0, issued - kAttnSlots); L < issued; ++L) {
                        const long long t0 = clock64();
                        while (!mbar_try_wait(bar(FULL + slot_of(L)), par_of(L)) && clock64() - t0 < 2000000) {}
                    }
                }
            } else if (pt < 128) {
            // (16-byte cp.async path: the first four producer warps gather, the others have nothing to do)
            // Up to three gathers are in flight and a load is posted (its FULL barrier signalled) once the two younger
            // ones have been issued -- unless the ring is full: then everything in flight is waited for and posted before
            // the warp blocks on the slot, so that the MMA side never waits for a load that has already landed.
            bool ok = true;
            int issued = 0, posted = 0;
            auto post_upto = [&](int n) {                 // loads [posted, n) have landed (the caller waited for them)
                fence_proxy_async();
                for (; posted < n; ++posted) mbar_arrive_warp(bar(FULL + slot_of(posted)));
            };
            for (int L = 0; L < 2 * n_tiles && ok; ++L) {
                const int i = L >> 1, is_v = L & 1, slot = slot_of(L);
                if (!__all_sync(0xffffffffu, mbar_test_wait(bar(EMPTY + slot), par_of(L) ^ 1))) {
                    cp_async_wait<0>();
                    post_upto(issued);
                    if (!mbar_wait(bar(EMPTY + slot), par_of(L) ^ 1, abort_s, status)) { ok = false; break; }
                }
                const __nv_bfloat16 *cache = is_v ? kv.v : kv.k, *blk = is_v ? v_blk : k_blk;
                uint8_t *tile = kv_s + slot * kTileBytes + (cchunk >> 3) * kHalfBytes;
#pragma unroll 4
                for (int it = 0; it < 16; ++it) {
                    const int r = r0 + 8 * it, t = i * kTile + r;
                    uint8_t *dst = tile + r * 128 + (((cchunk & 7) ^ (r & 7)) << 4);
                    const __nv_bfloat16 *src = nullptr;
                    if (t < n_cache) {
                        const int o = use_tab ? row_tab[t] : resolve(t);
                        if (o >= 0) src = cache + ((long long)o << 3) + cchunk * 8;
                    } else if (t < n_keys) {
                        src = blk + ((long long)z * kv.B + (t - blk_shift)) * kD + cchunk * 8;
                    }
                    if (src) cp_async_16(smem_u32(dst), src);
                    else *reinterpret_cast<uint4 *>(dst) = make_uint4(0, 0, 0, 0);
                }
                cp_async_commit();
                issued = L + 1;
                if (issued - posted > 2) {                // all but the two youngest groups are complete after this wait
                    cp_async_wait<2>();
                    post_upto(issued - 2);
                }
            }
            cp_async_wait<0>();
            if (ok) post_upto(issued);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issue (one lane)
        if (lane == 0) {
            const uint32_t idesc_qk = K8 ? idesc_e4m3_f32(kTile) : idesc_bf16_f32(kTile, false, false);   // S[128 rows][128 keys]
            const uint32_t idesc_qk_last = K8 ? idesc_e4m3_f32(last_cols) : idesc_bf16_f32(last_cols, false, false);
            const int nks_last = last_cols >> 4;                             // 16-key steps of the last tile's P V
            const uint32_t idesc_pv = idesc_bf16_f32(kD, false, true);       // O[128 rows][128 d], V is MN-major
            // The issuing thread runs in step with the tensor pipe (an MMA is accepted only as the previous one drains),
            // so whatever it executes between two MMAs is idle time of the pipe.  Hence: shared-memory descriptors are
            // a per-slot base plus a constant (same upper word for all of them: 1024-byte groups of eight rows, 128-byte
            // swizzle); ring positions advance without divisions; operand waits are taken before a batch of MMAs, not
            // inside it; the PV of a tile is issued in one go when P is already complete (half by half, with a commit
            // between, only when the softmax is the slower side); and key/value slots are handed back to the producer
            // by the softmax warpgroup that observes the next S (its commit covers every earlier MMA).
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            constexpr uint32_t kTileU = kTileBytes >> 4, kHalfU = kHalfBytes >> 4;     // 16-byte units
            auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
            const uint32_t q_lo = ((smem_u32(q_s) >> 4) & 0x3FFFu) | (1u << 16);           // K-major: 16-byte leading offset
            const uint32_t k_lo = ((smem_u32(kv_s) >> 4) & 0x3FFFu) | (1u << 16);
            const uint32_t v_lo = ((smem_u32(kv_s) >> 4) & 0x3FFFu) | (kHalfU << 16);       // MN-major: the two d-halves
            struct Ring {                                    // position of a load in the ring of slots, two loads per step
                int slot;
                uint32_t par;
                __device__ void next() {
                    slot += 2;
                    if (slot >= kAttnSlots) { slot -= kAttnSlots; par ^= 1u; }
                }
            };
            auto ring_at = [](int L) { return Ring{L % kAttnSlots, (uint32_t)((L / kAttnSlots) & 1)}; };
            // reg = which S/O region (and softmax warpgroup); the Q tile is reg with two M-tiles, tile 0 in tile-parity mode
            auto qk = [&](int slot, int reg, int tile) {
                const uint32_t a0 = q_lo + (tp ? 0u : (uint32_t)reg * kTileU), b0 = k_lo + (uint32_t)slot * kTileU;
                const uint32_t idesc = SPARSE && tile == n_tiles - 1 ? idesc_qk_last : idesc_qk;
                if (K8) {                                      // 32 one-byte elements of d per step, the row is one swizzle atom
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) umma_ss_f8(tmem_base + reg * 128, desc(a0 + ks * 2), desc(b0 + ks * 2), idesc, ks > 0);
                    return;
                }
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * kHalfU + (ks & 3) * 2;
                    umma_ss(tmem_base + reg * 128, desc(a0 + off), desc(b0 + off), idesc, ks > 0);
                }
            };
            // half 0: keys 0-63 of the tile, half 1: keys 64-127; 16 keys per step = 16 rows of 128 bytes in each d-half
            auto pv = [&](int slot, int reg, int half, uint32_t acc, int tile) {
                if (maps.lse_only) return;
                const uint32_t b0 = v_lo + (uint32_t)slot * kTileU;
                const int nks = SPARSE && tile == n_tiles - 1 ? nks_last : 8;
#pragma unroll
                for (int ks = half * 4; ks < half * 4 + 4; ++ks)
                    if (!SPARSE || ks < nks)
                        umma_ts(tmem_base + 256 + reg * 128, tmem_base + reg * 128 + ks * 8, desc(b0 + ks * (2048 >> 4)), idesc_pv, ks > 0 ? 1u : acc);
            };
            auto wait_full = [&](const Ring &r) { return mbar_wait(bar(FULL + r.slot), r.par, abort_s, status); };
            auto peek_p = [&](int reg, int ph) { return mbar_test_wait(bar(P_FULL + reg), ph); };
            // Looks at barriers ahead of time: the test is issued before a batch of MMAs and its result is used after it,
            // so its latency (about a hundred cycles even when the phase is complete) overlaps with the issue of the batch.
            auto peek_full = [&](const Ring &r) { return mbar_test_wait(bar(FULL + r.slot), r.par); };
            auto pv_tile = [&](int slot, int reg, int ph, uint32_t acc, bool p_ready, int tile) -> bool {
                if (p_ready || mbar_test_wait(bar(P_FULL + reg), ph)) {
                    tc_fence_after_sync();
                    pv(slot, reg, 0, acc, tile);
                    pv(slot, reg, 1, acc, tile);
                    return true;
                }
                if (!mbar_wait(bar(P_HALF + reg), ph, abort_s, status)) return false;
                tc_fence_after_sync();
                pv(slot, reg, 0, acc, tile);
                umma_commit(bar(PVH_DONE + reg));
                if (!mbar_wait(bar(P_FULL + reg), ph, abort_s, status)) return false;
                tc_fence_after_sync();
                pv(slot, reg, 1, acc, tile);
                return true;
            };
            // The reuse step is a handful of tiles long and latency-bound: there the slots go back by commits right after
            // their last MMA, which is sooner than the softmax warpgroup's wake-up.
            constexpr bool kCommitFrees = SPARSE;
            bool ok = mbar_wait(bar(Q_FULL), 0, abort_s, status);
            MAGE_STAMP(3);
            if (tp) {
                // tile i belongs to pipeline i & 1; its QK^T is issued two tiles ahead, right after the PV of tile i-2
                Ring rk = ring_at(0), rv = ring_at(1);
                for (int i = 0; ok && i < min(2, n_tiles); ++i, rk.next()) {
                    ok = wait_full(rk);
                    if (!ok) break;
                    tc_fence_after_sync();
                    qk(rk.slot, i, i);
                    umma_commit(bar(S_FULL + i));
                    if (kCommitFrees) umma_commit(bar(EMPTY + rk.slot));
                }
                rk = ring_at(4);
                for (int i = 0; ok && i < n_tiles; ++i, rk.next(), rv.next()) {
                    const int reg = i & 1, ph = (i >> 1) & 1;
                    if (!wait_full(rv)) break;
                    if (!pv_tile(rv.slot, reg, ph, i > 1 ? 1u : 0u, peek_p(reg, ph), i)) break;
                    // V(i) goes back by a commit of its own here: the next S of this pipeline needs K(i+2), and a gathering
                    // producer posts K(i+2) only after it has issued two more loads, the first of them into V(i)'s slot
                    umma_commit(bar(EMPTY + rv.slot));
                    if (i + 2 < n_tiles) {
                        if (!wait_full(rk)) break;
                        tc_fence_after_sync();
                        qk(rk.slot, reg, i + 2);
                        umma_commit(bar(S_FULL + reg));
                        if (kCommitFrees) umma_commit(bar(EMPTY + rk.slot));
                    }
                }
            } else {
                Ring rk = ring_at(0), rv = ring_at(1);
                if (ok) ok = wait_full(rk);
                MAGE_STAMP(4);
                if (ok) {
                    tc_fence_after_sync();
                    qk(rk.slot, 0, 0);
                    umma_commit(bar(S_FULL + 0));
                    qk(rk.slot, 1, 0);
                    umma_commit(bar(S_FULL + 1));
                    if (kCommitFrees) umma_commit(bar(EMPTY + rk.slot));
                }
                rk.next();
                bool v_ready = false, k_ready = false, p0_ready = false;          // looked at during the previous batch
                for (int i = 0; ok && i < n_tiles; ++i, rk.next(), rv.next()) {
                    const bool more = i + 1 < n_tiles;
                    const int ph = i & 1;
                    const uint32_t acc = i > 0 ? 1u : 0u;
                    if (!v_ready && !wait_full(rv)) break;
                    MAGE_STAMP(80 + i);
                    // (a gathered K(i+1) may land after P(i) is ready: the reuse step does not hold PV(i) back for it)
                    if (!SPARSE && more && !k_ready && !wait_full(rk)) break;
                    if (!pv_tile(rv.slot, 0, ph, acc, p0_ready, i)) break;
                    const bool p1_ready = peek_p(1, ph);
                    if (more) {
                        if (SPARSE) {
                            if (!wait_full(rk)) break;
                            tc_fence_after_sync();
                        }
                        qk(rk.slot, 0, i + 1);
                        umma_commit(bar(S_FULL + 0));
                    }
                    if (!pv_tile(rv.slot, 1, ph, acc, p1_ready, i)) break;
                    MAGE_STAMP(60 + i);
                    if (kCommitFrees) umma_commit(bar(EMPTY + rv.slot));
                    if (more) {
                        Ring rv1 = rv, rk1 = rk;
                        rv1.next();
                        rk1.next();
                        v_ready = peek_full(rv1);
                        k_ready = i + 2 < n_tiles && peek_full(rk1);
                        p0_ready = peek_p(0, ph ^ 1);
                        qk(rk.slot, 1, i + 1);
                        umma_commit(bar(S_FULL + 1));
                        if (kCommitFrees) umma_commit(bar(EMPTY + rk.slot));
                    }
                }
            }
            umma_commit(bar(O_DONE));
        }
    } else {
        // ------------------------------------------------------------------ softmax warpgroups
        const int mt = warp >> 2, w4 = warp & 3;
        if (mt < n_mt || tp) {
            const uint32_t lane_off = (uint32_t)(w4 * 32) << 16;
            const uint32_t tS = tmem_base + mt * 128 + lane_off, tO = tmem_base + 256 + mt * 128 + lane_off;
            const int first = tp ? mt : 0, stride = tp ? 2 : 1;      // tiles of this warpgroup: first, first + stride, ...
            const int row = w4 * 32 + lane, grow = rg * rgr + (tp ? 0 : mt * kTile) + row;
            const bool warp_has_rows = rg * rgr + (tp ? 0 : mt * kTile) + w4 * 32 < kv.M;
            float m_used = -INFINITY, l = 0.f;
            float pend_m = 0.f;          // reference the row wants to move to at the start of its next tile
            bool pending = false;
            const uint64_t c2 = pack2(scale_log2, scale_log2);
            bool ok = true;
            for (int i = first; i < n_tiles; i += stride) {
                const int ph = (tp ? i >> 1 : i) & 1;
                if (!__all_sync(0xffffffffu, mbar_wait(bar(S_FULL + mt), ph, abort_s, status))) { ok = false; break; }
                tc_fence_after_sync();
                if (tid == 0) MAGE_STAMP(10 + 2 * i);
                // S(i) complete means every MMA issued before it is complete too: K(i) and (two M-tiles) V(i-1), whose PV
                // was issued just before this QK^T, have been read for the last time; their slots go back to the producer.
                if (!SPARSE && w4 == 0 && lane == 0 && (tp || mt == 1)) {
                    mbar_arrive(bar(EMPTY + slot_of(2 * i)));
                    if (!tp && i >= 1) mbar_arrive(bar(EMPTY + slot_of(2 * i - 1)));
                }
                // phase of the "first half of PV accumulated" barrier before this tile's P exists (see the recovery path)
                const uint32_t pvh_cur = mbar_test_wait(bar(PVH_DONE + mt), 0) ? 1u : 0u;
                const int valid = min(kTile, n_keys - i * kTile);
                const int cols_here = SPARSE && i == n_tiles - 1 ? ((valid + 31) & ~31) : kTile;    // columns of S in use, by 32
                const int bad = SPARSE ? any_bad : tile_bad_s[i & 7];    // (rare) keys of this tile to leave out
                // Rescale O by f (rows that do not need it pass f = 1): no MMA touches this O between "S(i) complete"
                // (which implies PV(i-1) complete) and "P(i) ready".
                auto rescale_o = [&](float f) {
#pragma unroll 1
                    for (int c0 = 0; c0 < kD; c0 += 32) {
                        uint32_t r[32];
                        tmem_ld32(tO + c0, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * f);
                        tmem_st32(tO + c0, r);
                    }
                    tmem_wait_st();
                };
                // a warp whose 32 rows all lie beyond M (row padding of the last M-tile) only takes part in the hand-offs
                bool fast = valid == kTile && bad == 0, half_done = false;
                float tile_sum = 0.f;                      // this tile's part of l, relative to m_used as it stands after the tile
                if (warp_has_rows && fast && i == first) {
                    // first tile: the reference starts at the maximum of the row's first 32 logits; the sweep below moves it
                    // on lazily like any later rise (and redoes the tile on the careful path if the rest of the row lies
                    // more than 2^100 above it)
                    uint32_t r0[32];
                    tmem_ld32(tS, r0);
                    tmem_wait_ld(r0);
                    float m0 = __uint_as_float(r0[0]);
#pragma unroll
                    for (int e = 1; e < 32; ++e) m0 = fmaxf(m0, __uint_as_float(r0[e]));
                    m_used = m0 * scale_log2;
                }
                if (warp_has_rows && fast) {
                    // ---- common case: one sweep over S with the reference maximum carried over from earlier tiles.
                    // exp2(x - m_used) stays representable as long as x - m_used < 100, so the true maximum is only
                    // tracked (to move the reference lazily, at the next tile) and checked against that limit.
                    if (__any_sync(0xffffffffu, pending)) {
                        const float f = pending ? ex2(m_used - pend_m) : 1.f;
                        rescale_o(f);
                        l *= f;
                        if (pending) m_used = pend_m;
                        pending = false;
                    }
                    uint64_t neg_m2 = pack2(-m_used, -m_used);
                    uint64_t l2a = pack2(0.f, 0.f), l2b = l2a;
                    float mx = -INFINITY;
                    // 32 columns of S -> 16 packed bf16 pairs of P, the row sum and the running maximum of x
                    auto chunk = [&](const uint32_t (&r)[32], uint32_t (&pk)[16]) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const uint64_t x2 = fma2(pack2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), c2, neg_m2);
                            float x0, x1;
                            unpack2(x2, x0, x1);
                            mx = max3(mx, x0, x1);
                            const float p0 = ex2(x0), p1 = ex2(x1);
                            if (e & 1) l2b = add2(l2b, pack2(p0, p1));
                            else l2a = add2(l2a, pack2(p0, p1));
                            pk[e] = pack_bf16x2(p0, p1);
                        }
                    };
                    uint32_t ra[32], rb[32], pa[16], pb[16];
                    // first half of the tile (keys 0-63): nothing is stored before its maximum has been checked, so S
                    // is still whole if the tile has to be redone on the careful path
                    tmem_ld32(tS, ra);
                    tmem_wait_ld(ra);
                    tmem_ld32(tS + 32, rb);
                    chunk(ra, pa);
                    tmem_wait_ld(rb);
                    tmem_ld32(tS + 64, ra);
                    chunk(rb, pb);
                    if (__any_sync(0xffffffffu, mx > 100.f)) {
                        tmem_wait_ld(ra);
                        fast = false;
                    } else {
                        tmem_st16(tS, pa);
                        tmem_st16(tS + 16, pb);
                        tmem_wait_ld(ra);
                        tmem_ld32(tS + 96, rb);
                        tmem_wait_st();
                        tc_fence_before_sync();
                        mbar_arrive_warp(bar(P_HALF + mt));    // the PV MMA may start on keys 0-63
                        half_done = true;
                        // second half (keys 64-127): its P lands on S columns 32-63, already consumed; its own S
                        // columns 64-127 are never overwritten
                        const float mx_first = mx;
                        mx = -INFINITY;
                        chunk(ra, pa);
                        tmem_wait_ld(rb);
                        chunk(rb, pb);
                        if (__any_sync(0xffffffffu, mx > 100.f)) {
                            // A jump of more than 2^100 inside the tile (never seen in practice; kept for correctness):
                            // wait until the first half's PV has been accumulated, move the reference, redo keys 64-127.
                            // (the issuing thread finds P incomplete, issues the first half and commits to this barrier,
                            // which otherwise is not signalled at all: wait for the phase seen at the start of the tile)
                            if (!__all_sync(0xffffffffu, mbar_wait(bar(PVH_DONE + mt), pvh_cur, abort_s, status))) { ok = false; break; }
                            tc_fence_after_sync();
                            float a0, a1, b0, b1;
                            unpack2(l2a, a0, a1);
                            unpack2(l2b, b0, b1);
                            // l2a/l2b hold first-half terms (valid) and second-half terms (overflowed): recompute both
                            const float m_new = fmaxf(m_used, m_used + fmaxf(mx, mx_first));
                            const float f = ex2(m_used - m_new);
                            rescale_o(f);
                            l *= f;
                            float l_first = 0.f;           // first-half row sum, recomputed from the stored bf16 P
#pragma unroll
                            for (int c0 = 0; c0 < 32; c0 += 16) {
                                uint32_t pr[16];
                                tmem_ld16(tS + c0, pr);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 16; ++e) l_first += __uint_as_float(pr[e] << 16) + __uint_as_float(pr[e] & 0xffff0000u);
                            }
                            l += l_first * f;
                            tile_sum = l_first * f;
                            m_used = m_new;
                            neg_m2 = pack2(-m_used, -m_used);
                            l2a = pack2(0.f, 0.f);
                            l2b = l2a;
                            mx = -INFINITY;
                            tmem_ld32(tS + 64, ra);
                            tmem_wait_ld(ra);
                            tmem_ld32(tS + 96, rb);
                            chunk(ra, pa);
                            tmem_wait_ld(rb);
                            chunk(rb, pb);
                            mx = 0.f;
                        } else {
                            mx = fmaxf(mx, mx_first);
                        }
                        float a0, a1, b0, b1;
                        unpack2(l2a, a0, a1);
                        unpack2(l2b, b0, b1);
                        l += (a0 + a1) + (b0 + b1);
                        tile_sum += (a0 + a1) + (b0 + b1);
                        if (mx > kRescaleThreshold) { pending = true; pend_m = m_used + mx; }
                        tmem_st16(tS + 32, pa);
                        tmem_st16(tS + 48, pb);
                    }
                }
                if (warp_has_rows && !fast) {
                    // ---- careful path (first tile, ragged last tile, or a jump of the maximum by more than 2^100):
                    // find the tile's maximum first, move the reference if it grew, then exponentiate.
                    // bits of the 32 columns from c0 on that take part: inside the tile's valid keys and not left out
                    auto cols_ok = [&](int c0) -> uint32_t {
                        uint32_t okm = valid - c0 >= 32 ? 0xffffffffu : (valid - c0 <= 0 ? 0u : (1u << (valid - c0)) - 1u);
                        if (bad) {
                            if (!SPARSE) {
                                if ((bad >> (c0 >> 6)) & 1) okm = 0u;
                            } else {
                                okm &= ~sparse_bad_cols(use_tab ? row_tab : nullptr, indices + (long long)z * k + key_off, i * kTile + c0, n_cache, N,
                                                        kv.page_size ? kv.block_table + (long long)p * kv.max_pages : nullptr, kv.page_size, kv.num_pages);
                            }
                        }
                        return okm;
                    };
                    float mx = -INFINITY;
#pragma unroll 1
                    for (int c0 = 0; c0 < cols_here; c0 += 32) {
                        uint32_t r[32];
                        tmem_ld32(tS + c0, r);
                        tmem_wait_ld();
                        const uint32_t okm = cols_ok(c0);
                        if (okm == 0xffffffffu) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]));
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if ((okm >> e) & 1u) mx = fmaxf(mx, __uint_as_float(r[e]));
                        }
                    }
                    // (a tile all of whose keys are left out has no maximum: a finite stand-in far below any logit)
                    float target = mx == -INFINITY ? -1e30f : mx * scale_log2;
                    if (pending) target = fmaxf(target, pend_m);
                    if (i == first) {
                        m_used = target;
                    } else {
                        const bool need = pending || target > m_used + kRescaleThreshold;
                        if (__any_sync(0xffffffffu, need)) {
                            const float m_new = need ? fmaxf(target, m_used) : m_used;
                            const float f = ex2(m_used - m_new);
                            rescale_o(f);
                            l *= f;
                            m_used = m_new;
                        }
                    }
                    pending = false;
                    const float neg_m = -m_used;
                    float l0 = 0.f, l1 = 0.f;
#pragma unroll 1
                    for (int c0 = 0; c0 < cols_here; c0 += 32) {
                        uint32_t r[32], pk[16];
                        tmem_ld32(tS + c0, r);
                        tmem_wait_ld();
                        const uint32_t okm = cols_ok(c0);
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            float p0 = ex2(fmaf(__uint_as_float(r[2 * e]), scale_log2, neg_m));
                            float p1 = ex2(fmaf(__uint_as_float(r[2 * e + 1]), scale_log2, neg_m));
                            if (okm != 0xffffffffu) {
                                if (!((okm >> (2 * e)) & 1u)) p0 = 0.f;
                                if (!((okm >> (2 * e + 1)) & 1u)) p1 = 0.f;
                            }
                            l0 += p0;
                            l1 += p1;
                            pk[e] = pack_bf16x2(p0, p1);
                        }
                        tmem_st16(tS + (c0 >> 1), pk);
                    }
                    l += l0 + l1;
                    tile_sum = l0 + l1;
                }
                if (!SPARSE && maps.rowsum != nullptr && !blk_chunk && grow < kv.M)
                    maps.rowsum[((size_t)z * maps.rowsum_tiles + (j_begin / kTile + i)) * plan.Mw + grow] = make_float2(tile_sum, m_used);
                tmem_wait_st();
                if (!SPARSE && valid != kTile && (tp || mt == 0)) {
                    // Last tile of the prefix: cache rows past the end may hold anything (even NaN patterns), and
                    // 0 * NaN would poison O.  Zero those V rows in shared memory before the PV MMA may start.
                    const int Lv = 2 * i + 1;
                    if (!__all_sync(0xffffffffu, mbar_wait(bar(FULL + slot_of(Lv)), par_of(Lv), abort_s, status))) { ok = false; break; }
                    if (row >= valid) {
                        uint8_t *vrow = kv_s + slot_of(Lv) * kTileBytes + row * 128;
#pragma unroll
                        for (int q4 = 0; q4 < 8; ++q4) {
                            *reinterpret_cast<uint4 *>(vrow + q4 * 16) = make_uint4(0, 0, 0, 0);
                            *reinterpret_cast<uint4 *>(vrow + kHalfBytes + q4 * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }
                    fence_proxy_async();
                }
                tc_fence_before_sync();
                if (!half_done) mbar_arrive_warp(bar(P_HALF + mt));
                mbar_arrive_warp(bar(P_FULL + mt));
                if (tid == 0) MAGE_STAMP(11 + 2 * i);
            }
            // Tile-parity mode: warpgroup 1 publishes its (reference, sum) and is done; warpgroup 0 folds the second
            // accumulator (same TMEM lanes, columns + 128) into its own while it writes the result.  The spare Q tile
            // holds the published pairs.
            float2 *pub = reinterpret_cast<float2 *>(q_s + kTileBytes);
            const bool merge = tp && n_tiles > 1;
            float w0 = 1.f, w1 = 0.f;
            if (tp && mt == 1) {
                if (ok && merge) {
                    pub[row] = make_float2(m_used, l);
                    __threadfence_block();
                    mbar_arrive_warp(bar(PUB));
                }
                ok = false;                                  // nothing to write
            }
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(O_DONE), 0, abort_s, status));
            if (ok && merge) ok = __all_sync(0xffffffffu, mbar_wait(bar(PUB), 0, abort_s, status));
            if (tid == 0) MAGE_STAMP(30);
            if (ok) {
                tc_fence_after_sync();
                const bool row_ok = grow < kv.M;
                if (merge) {
                    const float2 o = pub[row];
                    const float m_all = fmaxf(m_used, o.x);
                    w0 = ex2(m_used - m_all);
                    w1 = ex2(o.x - m_all);
                    l = l * w0 + o.y * w1;
                    m_used = m_all;
                }
                auto load_o = [&](int c0, uint32_t (&r)[32]) {
                    tmem_ld32(tO + c0, r);
                    if (merge) {
                        uint32_t q[32];
                        tmem_ld32(tO + 128 + c0, q);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            r[e] = __float_as_uint(fmaf(__uint_as_float(q[e]), w1, __uint_as_float(r[e]) * w0));
                    } else {
                        tmem_wait_ld();
                    }
                };
                // A thread holds a row of O, so a store straight from registers would put 16 bytes into each of 32
                // different rows per instruction.  The rows go through shared memory instead (the key/value ring is idle
                // now; 64 fp32 or 128 bf16 columns at a time, rows padded by 16 bytes against bank conflicts) and leave as
                // whole 256-byte pieces, two rows per instruction.
                constexpr int kStageRow = 256 + 16;
                uint8_t *stg = kv_s + warp * (32 * kStageRow);
                const int row0 = rg * rgr + (tp ? 0 : mt * kTile) + w4 * 32;              // first row of this warp
                const int rows_ok = min(32, kv.M - row0);                                   // may be <= 0
                auto flush = [&](uint8_t *dst_row0, size_t dst_pitch) {                     // 32 staged rows of 256 bytes -> global
                    __syncwarp();
#pragma unroll 4
                    for (int it = 0; it < 16; ++it) {
                        const int rr = it * 2 + (lane >> 4), cb = (lane & 15) * 16;
                        const uint4 v = *reinterpret_cast<const uint4 *>(stg + rr * kStageRow + cb);
                        if (rr < rows_ok) *reinterpret_cast<uint4 *>(dst_row0 + (size_t)rr * dst_pitch + cb) = v;
                    }
                    __syncwarp();
                };
                auto store_partial = [&](float *po_row0, float *pml_row) {                  // unnormalised O, then (m, l)
#pragma unroll 1
                    for (int c0 = 0; c0 < (maps.lse_only ? 0 : kD); c0 += 64) {
#pragma unroll 1
                        for (int c1 = 0; c1 < 64; c1 += 32) {
                            uint32_t r[32];
                            load_o(c0 + c1, r);
#pragma unroll
                            for (int e = 0; e < 32; e += 4)
                                *reinterpret_cast<uint4 *>(stg + lane * kStageRow + (c1 + e) * 4) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
                        }
                        flush(reinterpret_cast<uint8_t *>(po_row0 + c0), (size_t)kD * 4);
                    }
                    if (row_ok) {
                        pml_row[0] = m_used;
                        pml_row[1] = l;
                    }
                };
                if (!SPARSE) {
                    const size_t item = (size_t)z * (plan.n_chunks + 1) + chunk;
                    store_partial(ws + plan.off_part_o + (item * plan.Mw + row0) * kD, ws + plan.off_part_ml + (item * plan.Mw + grow) * 2);
                } else if (gridDim.x > 1) {
                    const size_t item = (size_t)z * gridDim.x + chunk;
                    store_partial(ws + plan.off_sparse_o + (item * plan.Mw + row0) * kD, ws + plan.off_sparse_ml + (item * plan.Mw + grow) * 2);
                } else {
                    const float inv = 1.f / l;
#pragma unroll 1
                    for (int c0 = 0; c0 < kD; c0 += 32) {
                        uint32_t r[32];
                        load_o(c0, r);
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
                            v.y = pack_bf16x2(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
                            v.z = pack_bf16x2(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
                            v.w = pack_bf16x2(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
                            *reinterpret_cast<uint4 *>(stg + lane * kStageRow + (c0 + e) * 2) = v;
                        }
                    }
                    __nv_bfloat16 *po_row0 = out + ((long long)(p * kv.H_q + h * kv.G) * kv.B + row0) * kD;
                    flush(reinterpret_cast<uint8_t *>(po_row0), (size_t)kD * 2);
                }
            }
        }
    }
    if (tid == 0) MAGE_STAMP(31);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    if (tid == 0) MAGE_STAMP(32);
    MAGE_CLK(127);
}

// Merge of a reuse step that was split over n_split CTAs per KV head: one warp per query row, fixed order.
__global__ void __launch_bounds__(128) sparse_combine_kernel(KvView kv, Plan plan, int n_split, int k, const int *__restrict__ k_eff_arr,
                                                             const float *__restrict__ ws, __nv_bfloat16 *__restrict__ out) {
    ptx::pdl_wait();
    ptx::pdl_launch_dependents();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= kv.P * kv.H_kv * kv.M) return;
    const int z = warp / kv.M, r = warp % kv.M, p = z / kv.H_kv, h = z % kv.H_kv;
    const int n_keys = min(max(k_eff_arr[p], 0), k) + kv.B;
    const int tiles_all = (n_keys + kTile - 1) / kTile, per = (tiles_all + n_split - 1) / n_split;
    const int used = (tiles_all + per - 1) / per;               // splits that had work
    const float *ml = ws + plan.off_sparse_ml, *po = ws + plan.off_sparse_o;
    const size_t item0 = (size_t)z * n_split;
    // lane c holds split c's (m, l) (at most 32 splits); maximum and sum are warp reductions in a fixed order, the weights
    // travel by shuffle and four partial rows are in flight per lane
    float m_c = -INFINITY, l_c = 0.f;
    if (lane < used) {
        const float2 e = *reinterpret_cast<const float2 *>(ml + ((item0 + lane) * plan.Mw + r) * 2);
        m_c = e.x;
        l_c = e.y;
    }
    float m_all = m_c;
#pragma unroll
    for (int w = 16; w; w >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, w));
    const float w_c = lane < used ? exp2f(m_c - m_all) : 0.f;
    float l_all = l_c * w_c;
#pragma unroll
    for (int w = 16; w; w >>= 1) l_all += __shfl_xor_sync(0xffffffffu, l_all, w);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c0 = 0; c0 < used; c0 += 4) {
        float4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            v[q] = c0 + q < used ? *reinterpret_cast<const float4 *>(po + ((item0 + c0 + q) * plan.Mw + r) * kD + lane * 4)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float w = __shfl_sync(0xffffffffu, w_c, (c0 + q) & 31);
            acc.x = fmaf(v[q].x, w, acc.x); acc.y = fmaf(v[q].y, w, acc.y); acc.z = fmaf(v[q].z, w, acc.z); acc.w = fmaf(v[q].w, w, acc.w);
        }
    }
    const float inv = 1.f / l_all;
    __nv_bfloat16 *dst = out + ((long long)(p * kv.H_q + h * kv.G) * kv.B + r) * kD + lane * 4;
    __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), b = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<unsigned *>(&a), *reinterpret_cast<unsigned *>(&b));
}

}  // namespace tc
}  // namespace mage

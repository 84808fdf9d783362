// Per-KV-head exact Top-k of the block scores (Algorithm 1, select stream; Eq. 4) by radix select.
#pragma once
#include "common.cuh"

namespace mage {

constexpr int kTopkThreads = 1024;

// Order-preserving map from fp32 bit patterns to unsigned integers (larger float -> larger key).
__device__ __forceinline__ unsigned float_order_key(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One CTA per (problem, KV head).
//  1. three radix passes (11 + 11 + 10 key bits from the top, shared-memory histograms) find the k_eff-th largest key T
//     and how many entries equal to T are still needed;
//  2. one ordered pass emits every position with key > T and the first `need_eq` positions with key == T,
//     placed by a block-wide prefix sum, so the output is ascending and ties go to the smaller position.
// kth_out (optional, [P*H_kv]): the k_eff-th largest score of the row, or 0 when the row has no more than k entries.
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float *__restrict__ scores,
                                                            const int *__restrict__ seq_lens, int H_kv, int N_max,
                                                            int k, int *__restrict__ indices, int *__restrict__ k_eff_out,
                                                            float *__restrict__ kth_out = nullptr) {
    __shared__ unsigned hist4[4][2048];
    __shared__ unsigned hist[32];
    __shared__ unsigned warp_tot[32];
    __shared__ unsigned sel_digit, sel_need;

    const int z = blockIdx.x, p = z / H_kv, h = z % H_kv, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int N = seq_lens ? seq_lens[p] : N_max;
    N = N < 0 ? 0 : (N > N_max ? N_max : N);
    const int k_eff = k < N ? k : N;
    const float *s = scores + (size_t)z * N_max;
    int *out = indices + (size_t)z * k;
    if (h == 0 && tid == 0) k_eff_out[p] = k_eff;
    if (kth_out && tid == 0) kth_out[z] = 0.f;           // rows with no more than k entries have no threshold
    for (int t = k_eff + tid; t < k; t += kTopkThreads) out[t] = -1;
    if (k_eff == 0) return;
    if (k_eff == N) {
        for (int j = tid; j < N; j += kTopkThreads) out[j] = j;
        return;
    }

    const bool vec_ok = (reinterpret_cast<uintptr_t>(s) & 15) == 0;
    // Visit the row 16 elements per thread and iteration, all four 16-byte loads issued before any is used.
    auto for_each8 = [&](auto &&body) {
        for (int base = 0; base < N; base += kTopkThreads * 16) {
            float v[16];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const int j = base + q4 * kTopkThreads * 4 + tid * 4;
                if (vec_ok && j + 3 < N) {
                    const float4 f = *reinterpret_cast<const float4 *>(s + j);
                    v[q4 * 4 + 0] = f.x; v[q4 * 4 + 1] = f.y; v[q4 * 4 + 2] = f.z; v[q4 * 4 + 3] = f.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) v[q4 * 4 + e] = j + e < N ? s[j + e] : 0.f;
                }
            }
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int j = base + (e >> 2) * kTopkThreads * 4 + tid * 4 + (e & 3);
                if (j < N) body(float_order_key(v[e]));
            }
        }
    };

    // Three radix passes over the 32 key bits, 11 + 11 + 10 bits from the top: each reads the row once (the launch is bound
    // by L2 bandwidth times the number of passes, so fewer, wider digits beat a min/max pre-pass plus 8-bit digits).  Keys of
    // one head crowd into a few values of the first digit (same sign, neighbouring exponents), so the histogram is kept
    // in four copies (warp & 3) to spread the shared-memory atomics; after the first pass only keys that match the prefix
    // found so far touch it.
    unsigned prefix = 0u, mask = 0u, need = (unsigned)k_eff;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int lo = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const unsigned dmask = pass == 2 ? 1023u : 2047u;
        for (int t = tid; t < 4 * 2048; t += kTopkThreads) (&hist4[0][0])[t] = 0;
        __syncthreads();
        unsigned *my_hist = hist4[warp & 3];
        for_each8([&](unsigned key) {
            if ((key & mask) == prefix) atomicAdd(&my_hist[(key >> lo) & dmask], 1u);
        });
        __syncthreads();
        // number of candidates with digit >= d, for the two digits 2 * tid and 2 * tid + 1 of this thread: suffix sums by
        // shuffles inside the warp (64 digits), then the totals of the warps above
        const unsigned c0 = hist4[0][2 * tid] + hist4[1][2 * tid] + hist4[2][2 * tid] + hist4[3][2 * tid];
        const unsigned c1 = hist4[0][2 * tid + 1] + hist4[1][2 * tid + 1] + hist4[2][2 * tid + 1] + hist4[3][2 * tid + 1];
        unsigned v = c0 + c1;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned dn = __shfl_down_sync(0xffffffffu, v, off);
            if (lane + off < 32) v += dn;
        }
        if (lane == 0) warp_tot[warp] = v;
        __syncthreads();
        unsigned above = 0;
        for (int w = warp + 1; w < 32; ++w) above += warp_tot[w];
        const unsigned ge0 = v + above, ge1 = ge0 - c0, ge2 = ge1 - c1;       // candidates with digit >= 2t, >= 2t+1, >= 2t+2
        if (ge1 >= need && ge2 < need) { sel_digit = 2 * tid + 1; sel_need = need - ge2; }
        else if (ge0 >= need && ge1 < need) { sel_digit = 2 * tid; sel_need = need - ge1; }
        __syncthreads();
        prefix |= sel_digit << lo;
        mask |= dmask << lo;
        need = sel_need;
        __syncthreads();
    }
    const unsigned T = prefix, need_eq = need;
    if (kth_out && tid == 0) kth_out[z] = __uint_as_float((T & 0x80000000u) ? (T & 0x7fffffffu) : ~T);

    // Ordered emit.  A stretch of 32 x span entries at a time (span = 4096, less for short rows so that every warp has a
    // share): warp w owns entries [w * span, (w + 1) * span) of the stretch, lane l the four entries at 128 * i + 4 * l of
    // each of its span / 128 <= 32 rounds (coalesced 16-byte loads, eight in flight).  The
    // scores are read once: each lane keeps one "greater" and one "equal" bit per entry (2 x 128 bits), the warps' counts
    // meet in one block-wide prefix sum, and the positions are then written from the bit masks; rounds in which no lane of
    // the warp holds a selected entry (almost all of them: k of N entries are selected) cost one ballot.
    auto load4 = [&](int j_first, float (&v)[4]) {
        if (vec_ok && j_first + 3 < N) {
            const float4 f = *reinterpret_cast<const float4 *>(s + j_first);
            v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = j_first + e < N ? s[j_first + e] : 0.f;
        }
    };
    const int kWarpSpan = min(4096, ((N + 31) / 32 + 127) / 128 * 128), kStretch = 32 * kWarpSpan, rounds = kWarpSpan / 128;
    unsigned run_gt = 0, run_eq = 0;                     // selected entries before the current stretch
    for (int base = 0; base < N; base += kStretch) {
        const int w0 = base + warp * kWarpSpan;
        unsigned gt_bits[4] = {0, 0, 0, 0}, eq_bits[4] = {0, 0, 0, 0};
        if (w0 < N) {
#pragma unroll
            for (int i0 = 0; i0 < 32; i0 += 8) {
                float v[8][4];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int j_first = w0 + (i0 + u) * 128 + lane * 4;
                    if (i0 + u < rounds && j_first < N) load4(j_first, v[u]);
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int j_first = w0 + (i0 + u) * 128 + lane * 4;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (i0 + u < rounds && j_first + e < N) {
                            const unsigned key = float_order_key(v[u][e]);
                            if (key > T) gt_bits[i0 >> 3] |= 1u << (u * 4 + e);
                            else if (key == T) eq_bits[i0 >> 3] |= 1u << (u * 4 + e);
                        }
                    }
                }
            }
        }
        unsigned n_gt = __popc(gt_bits[0]) + __popc(gt_bits[1]) + __popc(gt_bits[2]) + __popc(gt_bits[3]);
        unsigned n_eq = __popc(eq_bits[0]) + __popc(eq_bits[1]) + __popc(eq_bits[2]) + __popc(eq_bits[3]);
        n_gt = __reduce_add_sync(0xffffffffu, n_gt);
        n_eq = __reduce_add_sync(0xffffffffu, n_eq);
        if (lane == 0) { warp_tot[warp] = n_gt; hist[warp] = n_eq; }
        __syncthreads();
        // exclusive prefix of the warps' counts (every warp computes the one it needs) and the stretch totals
        unsigned wg = warp_tot[lane], we = hist[lane];
        unsigned gt_before = run_gt + __reduce_add_sync(0xffffffffu, lane < warp ? wg : 0u);
        unsigned eq_before = run_eq + __reduce_add_sync(0xffffffffu, lane < warp ? we : 0u);
        run_gt += __reduce_add_sync(0xffffffffu, wg);
        run_eq += __reduce_add_sync(0xffffffffu, we);
        if (n_gt + n_eq != 0) {
#pragma unroll 1
            for (int i = 0; i < rounds; ++i) {
                const unsigned ng = (gt_bits[i >> 3] >> ((i & 7) * 4)) & 15u, ne = (eq_bits[i >> 3] >> ((i & 7) * 4)) & 15u;
                if (__ballot_sync(0xffffffffu, (ng | ne) != 0u) == 0u) continue;
                const unsigned packed = ((unsigned)__popc(ng) << 16) | (unsigned)__popc(ne);
                unsigned incl = packed;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const unsigned up = __shfl_up_sync(0xffffffffu, incl, off);
                    if (lane >= off) incl += up;
                }
                const unsigned tot = __shfl_sync(0xffffffffu, incl, 31), excl = incl - packed;
                unsigned g = gt_before + (excl >> 16), q = eq_before + (excl & 0xffffu);
                const int j_first = w0 + i * 128 + lane * 4;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (ng & (1u << e)) {
                        out[g + min(q, need_eq)] = j_first + e;
                        ++g;
                    } else if (ne & (1u << e)) {
                        if (q < need_eq) out[g + q] = j_first + e;
                        ++q;
                    }
                }
                gt_before += tot >> 16;
                eq_before += tot & 0xffffu;
            }
        }
        __syncthreads();                                  // warp_tot / hist are rewritten by the next stretch
    }
}


// ------------------------------------------------------------------------------------------------------------
// The same selection with a cluster of eight CTAs per (problem, KV head), for long rows: CTA c owns the c-th eighth of
// the row and keeps it in shared memory, so the scores are read from L2 once instead of once per pass, by eight SMs
// instead of one.  The CTAs meet through distributed shared memory (plain remote loads and stores): per radix pass every
// CTA publishes its digit histogram in its own shared memory, one cluster barrier, and every CTA adds up the eight
// histograms and takes the same decision; before the ordered emit the CTAs exchange how many selected entries each holds.  Exact and deterministic like the single-CTA kernel, same output.
// ------------------------------------------------------------------------------------------------------------
constexpr int kTopkCluster = 8;
constexpr int kTopkSliceCap = 40960;                    // floats of a CTA's share kept in shared memory (160 KB)
constexpr size_t kTopkClusterSmem = 7 * 2048 * sizeof(unsigned) + (size_t)kTopkSliceCap * sizeof(float);

#ifdef MAGE_TIMING
__device__ unsigned long long g_topk_stamps[64];
#define TOPK_STAMP(i) do { if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_topk_stamps[i] = t_; } } while (0)
#else
#define TOPK_STAMP(i) ((void)0)
#endif

namespace cl {
__device__ __forceinline__ unsigned cta_rank() { unsigned r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ unsigned map_to(const void *smem_ptr, unsigned rank) {         // this CTA's address -> CTA `rank`'s
    unsigned a = static_cast<unsigned>(__cvta_generic_to_shared(smem_ptr)), r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    return r;
}
__device__ __forceinline__ unsigned ld_u32(unsigned addr) { unsigned v; asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory"); return v; }
// every thread of every CTA of the cluster; orders the remote accesses before it against those after it
__device__ __forceinline__ void sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
}  // namespace cl

__global__ void __launch_bounds__(kTopkThreads) topk_cluster_kernel(const float *__restrict__ scores, const int *__restrict__ seq_lens,
                                                                    int H_kv, int N_max, int k, int *__restrict__ indices,
                                                                    int *__restrict__ k_eff_out) {
    extern __shared__ __align__(16) unsigned char dyn_s[];
    unsigned (*hist4)[2048] = reinterpret_cast<unsigned (*)[2048]>(dyn_s);                                // [4][2048]
    unsigned (*mine)[2048] = reinterpret_cast<unsigned (*)[2048]>(dyn_s + 4 * 2048 * sizeof(unsigned));   // [3][2048]: this CTA's digit counts of each pass, read by its peers
    float *slice_s = reinterpret_cast<float *>(dyn_s + 7 * 2048 * sizeof(unsigned));
    __shared__ unsigned merged[3][256];                  // digits [256 c, 256 c + 256) summed over the cluster, per pass
    __shared__ unsigned counts[2];                       // selected (greater, equal) entries this CTA holds, read by the CTAs after it
    __shared__ unsigned hist[32], warp_tot[32];
    __shared__ unsigned sel_digit, sel_need;

    TOPK_STAMP(0);
    const unsigned c = cl::cta_rank();
    const int z = blockIdx.y, p = z / H_kv, h = z % H_kv, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int N = seq_lens ? seq_lens[p] : N_max;
    N = N < 0 ? 0 : (N > N_max ? N_max : N);
    const int k_eff = k < N ? k : N;
    const float *row = scores + (size_t)z * N_max;
    int *out = indices + (size_t)z * k;
    // the trivial cases are the same for every CTA of the cluster: all of them leave before the first cluster barrier
    if (k_eff == 0 || k_eff == N) {
        if (c == 0) {
            if (h == 0 && tid == 0) k_eff_out[p] = k_eff;
            for (int t = tid; t < k; t += kTopkThreads) out[t] = t < k_eff ? t : -1;
        }
        return;
    }
    if (c == 0) {
        if (h == 0 && tid == 0) k_eff_out[p] = k_eff;
        for (int t = k_eff + tid; t < k; t += kTopkThreads) out[t] = -1;
    }
    // this CTA's share [lo, lo + n) of the row, a multiple of four entries long
    const int share = (((N + kTopkCluster - 1) / kTopkCluster) + 3) & ~3;
    const int lo = min(N, (int)c * share), n = min(N, lo + share) - lo;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
    const bool cached = share <= kTopkSliceCap;
    if (cached) {
        for (int j = tid * 4; j < n; j += kTopkThreads * 4) {
            if (vec_ok && j + 3 < n) {
                *reinterpret_cast<float4 *>(slice_s + j) = *reinterpret_cast<const float4 *>(row + lo + j);
            } else {
                for (int e = 0; e < 4 && j + e < n; ++e) slice_s[j + e] = row[lo + j + e];
            }
        }
    }
    TOPK_STAMP(1);
    const float *s = cached ? slice_s : row + lo;
    const bool s_vec = cached || vec_ok;
    __syncthreads();
    TOPK_STAMP(2);

    auto for_each = [&](auto &&body) {
        for (int base = 0; base < n; base += kTopkThreads * 16) {
            float v[16];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const int j = base + q4 * kTopkThreads * 4 + tid * 4;
                if (s_vec && j + 3 < n) {
                    const float4 f = *reinterpret_cast<const float4 *>(s + j);
                    v[q4 * 4 + 0] = f.x; v[q4 * 4 + 1] = f.y; v[q4 * 4 + 2] = f.z; v[q4 * 4 + 3] = f.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) v[q4 * 4 + e] = j + e < n ? s[j + e] : 0.f;
                }
            }
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int j = base + (e >> 2) * kTopkThreads * 4 + tid * 4 + (e & 3);
                if (j < n) body(float_order_key(v[e]));
            }
        }
    };

    unsigned prefix = 0u, mask = 0u, need = (unsigned)k_eff;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int lob = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const unsigned dmask = pass == 2 ? 1023u : 2047u;
        for (int t = tid; t < 4 * 2048; t += kTopkThreads) (&hist4[0][0])[t] = 0;
        __syncthreads();
        unsigned *my_hist = hist4[warp & 3];
        for_each([&](unsigned key) {
            if ((key & mask) == prefix) atomicAdd(&my_hist[(key >> lob) & dmask], 1u);
        });
        __syncthreads();
        TOPK_STAMP(3 + 4 * pass);
        // this CTA's counts of the digits 2 * tid, 2 * tid + 1 are published in its own shared memory; after the barrier every
        // CTA reads all eight CTAs' counts of its threads' digits (sixteen remote loads in flight at once) and adds them up
        mine[pass][2 * tid] = hist4[0][2 * tid] + hist4[1][2 * tid] + hist4[2][2 * tid] + hist4[3][2 * tid];
        mine[pass][2 * tid + 1] = hist4[0][2 * tid + 1] + hist4[1][2 * tid + 1] + hist4[2][2 * tid + 1] + hist4[3][2 * tid + 1];
        TOPK_STAMP(4 + 4 * pass);
        cl::sync_all();
        TOPK_STAMP(5 + 4 * pass);
        // two steps, so that a CTA makes 4096 remote loads per pass instead of 16384: CTA c adds up digits [256 c, 256 c + 256)
        // over the eight CTAs and publishes the sums; after a second barrier every thread fetches its two digits' sums
        if (tid < 256) {
            unsigned part[kTopkCluster];
#pragma unroll
            for (int cc = 0; cc < kTopkCluster; ++cc) part[cc] = cl::ld_u32(cl::map_to(&mine[pass][256 * c + tid], cc));
            unsigned sum = 0;
#pragma unroll
            for (int cc = 0; cc < kTopkCluster; ++cc) sum += part[cc];
            merged[pass][tid] = sum;
        }
        cl::sync_all();
        const unsigned owner = cl::map_to(&merged[pass][(2 * tid) & 255], (unsigned)(2 * tid) >> 8);
        const unsigned c0 = cl::ld_u32(owner), c1 = cl::ld_u32(owner + 4);
        unsigned v = c0 + c1;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned dn = __shfl_down_sync(0xffffffffu, v, off);
            if (lane + off < 32) v += dn;
        }
        if (lane == 0) warp_tot[warp] = v;
        __syncthreads();
        unsigned above = 0;
        for (int w = warp + 1; w < 32; ++w) above += warp_tot[w];
        const unsigned ge0 = v + above, ge1 = ge0 - c0, ge2 = ge1 - c1;
        if (ge1 >= need && ge2 < need) { sel_digit = 2 * tid + 1; sel_need = need - ge2; }
        else if (ge0 >= need && ge1 < need) { sel_digit = 2 * tid; sel_need = need - ge1; }
        __syncthreads();
        prefix |= sel_digit << lob;
        mask |= dmask << lob;
        need = sel_need;
        __syncthreads();
        TOPK_STAMP(6 + 4 * pass);
    }
    const unsigned T = prefix, need_eq = need;

    // Ordered emit.  Thread t owns 16 consecutive entries of each 16384-entry stretch of the share.  First sweep: how many
    // entries above / equal to the threshold the CTA holds, published for the CTAs after it; second sweep: a block-wide
    // prefix sum places each thread's entries.  Ties go to the smaller position: an equal entry is written only while
    // fewer than need_eq equal entries precede it in the row.
    auto masks_of = [&](int base, unsigned &gt, unsigned &eq) {
        gt = eq = 0;
        const int j0 = base + tid * 16;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            float v[4];
            const int j = j0 + q4 * 4;
            if (s_vec && j + 3 < n) {
                const float4 f = *reinterpret_cast<const float4 *>(s + j);
                v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) v[e] = j + e < n ? s[j + e] : 0.f;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (j + e < n) {
                    const unsigned key = float_order_key(v[e]);
                    gt |= (unsigned)(key > T) << (q4 * 4 + e);
                    eq |= (unsigned)(key == T) << (q4 * 4 + e);
                }
            }
        }
    };
    unsigned my_gt = 0, my_eq = 0;
    for (int base = 0; base < n; base += kTopkThreads * 16) {
        unsigned gt, eq;
        masks_of(base, gt, eq);
        my_gt += __popc(gt);
        my_eq += __popc(eq);
    }
    my_gt = __reduce_add_sync(0xffffffffu, my_gt);
    my_eq = __reduce_add_sync(0xffffffffu, my_eq);
    if (lane == 0) { warp_tot[warp] = my_gt; hist[warp] = my_eq; }
    __syncthreads();
    if (warp == 0) {
        const unsigned g = __reduce_add_sync(0xffffffffu, warp_tot[lane]), e = __reduce_add_sync(0xffffffffu, hist[lane]);
        if (lane == 0) { counts[0] = g; counts[1] = e; }
    }
    TOPK_STAMP(20);
    cl::sync_all();
    TOPK_STAMP(21);
    unsigned run_gt = 0, run_eq = 0;                      // selected entries before this CTA's share
    for (unsigned cc = 0; cc < c; ++cc) {
        run_gt += cl::ld_u32(cl::map_to(&counts[0], cc));
        run_eq += cl::ld_u32(cl::map_to(&counts[1], cc));
    }
    for (int base = 0; base < n; base += kTopkThreads * 16) {
        unsigned gt, eq;
        masks_of(base, gt, eq);
        const unsigned packed = ((unsigned)__popc(gt) << 16) | (unsigned)__popc(eq);
        unsigned incl = packed;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        __syncthreads();                                  // warp_tot is free again
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        unsigned before = 0, total = 0;
        for (int w = 0; w < 32; ++w) {
            const unsigned wt = warp_tot[w];
            before += w < warp ? wt : 0u;
            total += wt;
        }
        const unsigned excl = before + incl - packed;
        unsigned g = run_gt + (excl >> 16), q = run_eq + (excl & 0xffffu);
        if (gt | eq) {
            const int j0 = lo + base + tid * 16;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                if (gt & (1u << e)) {
                    out[g + min(q, need_eq)] = j0 + e;
                    ++g;
                } else if (eq & (1u << e)) {
                    if (q < need_eq) out[g + q] = j0 + e;
                    ++q;
                }
            }
        }
        run_gt += total >> 16;
        run_eq += total & 0xffffu;
    }
    TOPK_STAMP(22);
    cl::sync_all();                                       // CTA 0's shared memory stays until every CTA has read it
    TOPK_STAMP(23);
}

}  // namespace mage

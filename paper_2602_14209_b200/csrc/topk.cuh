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
//  1. four 8-bit radix passes over the keys find the k_eff-th largest key T and how many entries equal to T
//     are still needed (histograms in shared memory, warp-aggregated atomics);
//  2. one ordered pass emits every position with key > T and the first `need_eq` positions with key == T,
//     placed by a block-wide prefix sum, so the output is ascending and ties go to the smaller position.
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float *__restrict__ scores,
                                                            const int *__restrict__ seq_lens, int H_kv, int N_max,
                                                            int k, int *__restrict__ indices, int *__restrict__ k_eff_out) {
    __shared__ unsigned hist[256];
    __shared__ unsigned suffix[257];
    __shared__ unsigned warp_tot[32];
    __shared__ unsigned sel_digit, sel_need;

    const int z = blockIdx.x, p = z / H_kv, h = z % H_kv, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int N = seq_lens ? seq_lens[p] : N_max;
    N = N < 0 ? 0 : (N > N_max ? N_max : N);
    const int k_eff = k < N ? k : N;
    const float *s = scores + (size_t)z * N_max;
    int *out = indices + (size_t)z * k;
    if (h == 0 && tid == 0) k_eff_out[p] = k_eff;
    for (int t = k_eff + tid; t < k; t += kTopkThreads) out[t] = -1;
    if (k_eff == 0) return;
    if (k_eff == N) {
        for (int j = tid; j < N; j += kTopkThreads) out[j] = j;
        return;
    }

    unsigned prefix = 0, mask = 0, need = (unsigned)k_eff;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int j0 = 0; j0 < N; j0 += kTopkThreads) {
            const int j = j0 + tid;
            unsigned key = 0;
            bool valid = j < N;
            if (valid) { key = float_order_key(s[j]); valid = (key & mask) == prefix; }
            const unsigned digit = (key >> shift) & 255u;
            const unsigned peers = __match_any_sync(0xffffffffu, valid ? digit : 256u + lane);
            if (valid && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
        }
        __syncthreads();
        // suffix[t] = number of candidates whose digit is >= t
        if (tid < 256) suffix[tid] = hist[tid];
        if (tid == 0) suffix[256] = 0;
        __syncthreads();
        for (int off = 1; off < 256; off <<= 1) {
            unsigned add = 0;
            if (tid < 256 && tid + off < 256) add = suffix[tid + off];
            __syncthreads();
            if (tid < 256) suffix[tid] += add;
            __syncthreads();
        }
        if (tid < 256 && suffix[tid] >= need && suffix[tid + 1] < need) {
            sel_digit = tid;
            sel_need = need - suffix[tid + 1];
        }
        __syncthreads();
        prefix |= sel_digit << shift;
        mask |= 255u << shift;
        need = sel_need;
        __syncthreads();
    }
    const unsigned T = prefix, need_eq = need;

    const bool vec_ok = (reinterpret_cast<uintptr_t>(s) & 15) == 0;
    unsigned run_gt = 0, run_eq = 0;
    for (int base = 0; base < N; base += kTopkThreads * 4) {
        const int j_first = base + tid * 4;
        float v[4];
        if (vec_ok && j_first + 3 < N) {
            const float4 f = *reinterpret_cast<const float4 *>(s + j_first);
            v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = j_first + e < N ? s[j_first + e] : 0.f;
        }
        unsigned gt = 0, eq = 0, is_gt = 0, is_eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (j_first + e < N) {
                const unsigned key = float_order_key(v[e]);
                if (key > T) { is_gt |= 1u << e; ++gt; }
                else if (key == T) { is_eq |= 1u << e; ++eq; }
            }
        }
        const unsigned packed = (gt << 16) | eq;        // a chunk holds 4096 entries, so neither half overflows
        unsigned incl = packed;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned w = warp_tot[lane], wi = w;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned up = __shfl_up_sync(0xffffffffu, wi, off);
                if (lane >= off) wi += up;
            }
            warp_tot[lane] = wi - w;                    // exclusive prefix of the warp totals
            if (lane == 31) suffix[0] = wi;             // chunk total
        }
        __syncthreads();
        const unsigned excl = incl - packed + warp_tot[warp];
        unsigned gt_before = run_gt + (excl >> 16), eq_before = run_eq + (excl & 0xffffu);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (is_gt & (1u << e)) {
                out[gt_before + min(eq_before, need_eq)] = j_first + e;
                ++gt_before;
            } else if (is_eq & (1u << e)) {
                if (eq_before < need_eq) out[gt_before + eq_before] = j_first + e;
                ++eq_before;
            }
        }
        const unsigned tot = suffix[0];
        run_gt += tot >> 16;
        run_eq += tot & 0xffffu;
        __syncthreads();
    }
}

}  // namespace mage

// Shared device-side definitions of libmage: the cache view, row addressing and small math helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mage.h"

namespace mage {

constexpr int kD = 128;              // head dimension (bf16 row = 256 bytes)
constexpr float kLog2e = 1.4426950408889634f;

// Device copy of the cache description (Algorithm 1's prefix cache C), plus derived sizes.
struct KvView {
    const __nv_bfloat16 *k, *v;
    long long stride_p, stride_h, stride_n;   // contiguous layout, in elements
    const int *block_table;                   // paged layout
    const int *seq_lens;                      // may be null
    int max_pages, num_pages, page_size;      // page_size 0 = contiguous
    int N_max;
    int P, H_q, H_kv, B, G, M;                // M = G * B query rows per KV head
};

__device__ __forceinline__ int seq_len_of(const KvView &kv, int p) {
    int n = kv.seq_lens ? kv.seq_lens[p] : kv.N_max;
    return n < 0 ? 0 : (n > kv.N_max ? kv.N_max : n);
}

// Element offset of cache row (p, h, j) from the K (or V) base; -1 and a status bit when the page id is bad.
__device__ __forceinline__ long long cache_row_offset(const KvView &kv, int p, int h, int j, unsigned *status) {
    if (kv.page_size == 0) return (long long)p * kv.stride_p + (long long)h * kv.stride_h + (long long)j * kv.stride_n;
    const int page = kv.block_table[(long long)p * kv.max_pages + j / kv.page_size];
    if (page < 0 || page >= kv.num_pages) {
        if (status) atomicOr(status, MAGE_DEV_BAD_PAGE);
        return -1;
    }
    return (((long long)page * kv.H_kv + h) * kv.page_size + (j % kv.page_size)) * (long long)kD;
}

__device__ __forceinline__ void bf16x8_to_float(const uint4 &raw, float *out) {
    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h2[i]);
        out[2 * i] = f.x;
        out[2 * i + 1] = f.y;
    }
}

// Workspace plan shared by the host entry points and the kernels (all sizes in elements of the named type).
struct Plan {
    int M, Mw;               // query rows per KV head, padded to a multiple of 128
    int chunk_len, n_chunks; // split of the prefix for the exact pass; item n_chunks is the block's own keys
    size_t off_part_o;       // float [P*H_kv][n_chunks+1][Mw][128]   unnormalised partial outputs
    size_t off_part_ml;      // float [P*H_kv][n_chunks+1][Mw][2]     (m, l) in the log2 domain
    size_t off_neg_lse;      // float [P*H_kv][Mw]                    -log2-sum-exp over the prefix, per row
    int sparse_split_max;    // most CTAs that may share one KV head's selected keys in the reuse step
    size_t off_sparse_o;     // float [P*H_kv][sparse_split_max][Mw][128]  partial outputs of a split reuse step
    size_t off_sparse_ml;    // float [P*H_kv][sparse_split_max][Mw][2]
    size_t total_bytes;      // whole workspace; exact_bytes covers what mage_exact_select touches
    size_t exact_bytes;
};

}  // namespace mage

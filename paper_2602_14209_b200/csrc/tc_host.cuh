// Host side of the tensor-core path: TMA tensor maps (built per call, passed by value as kernel parameters)
// and launch geometry.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "tc_kernels.cuh"

namespace mage {
namespace tc {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                   const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up through the runtime, so the library does not link against libcuda.
inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Tensor of `rank` dims (dim 0 = the 128-element head dimension), 128-byte swizzle.  eb = bytes per element: 2 = bf16, boxes
// of 64 x 64 (x 1 x 1) elements (a d-half); 1 = e4m3 codes moved as bytes, boxes of 128 x 64: a whole row is 128 bytes.
inline bool make_map(CUtensorMap *m, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides_bytes,
                     unsigned box_rows = 64, int eb = 2) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t box[4] = {eb == 1 ? 128u : 64u, box_rows, 1, 1}, estr[4] = {1, 1, 1, 1};
    if (dims[1] < 1) return false;
    return fn(m, eb == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), dims, strides_bytes, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows][128] row-major matrix (queries, or the block's own keys / values).
inline bool make_rows_map(CUtensorMap *m, const void *base, long long rows, int eb = 2) {
    cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows}, str[1] = {(cuuint64_t)kD * eb};
    return make_map(m, base, 2, dims, str, 64, eb);
}

// Queries as (d, G*B rows of one KV head, P*H_kv heads): a 128-row tile that reaches past the head's last query row
// is filled with zeros there instead of the next head's rows (no work for the multipliers, nothing to mask later).
inline bool make_group_rows_map(CUtensorMap *m, const void *base, long long groups, int rows_per_group, int eb = 2) {
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)rows_per_group, (cuuint64_t)groups};
    cuuint64_t str[2] = {(cuuint64_t)kD * eb, (cuuint64_t)rows_per_group * kD * eb};
    return make_map(m, base, 3, dims, str, 64, eb);
}

// Row gather of the reuse step: the same memory as a flat list of 256-byte rows with one pitch, fetched one row
// (64 x 1 box per half) at a time; each row lands swizzled exactly as it would inside a 64-row box.
inline bool make_row_gather_map(CUtensorMap *m, const void *base, long long rows, long long pitch_elems, int eb = 2) {
    if (rows < 1 || rows > 0x7fffffffLL) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows}, str[1] = {(cuuint64_t)pitch_elems * eb};
    return make_map(m, base, 2, dims, str, 1, eb);
}
// Number of rows and pitch of the cache seen that way; false when the strides do not form one pitch.
inline bool cache_as_rows(const mage_kv_t *kv, long long *rows, long long *pitch) {
    if (kv->page_size != 0) {
        *rows = (long long)kv->num_pages * kv->H_kv * kv->page_size;
        *pitch = kD;
        return true;
    }
    if (kv->stride_n < kD || kv->stride_h % kv->stride_n || kv->stride_p % kv->stride_n) return false;
    *pitch = kv->stride_n;
    *rows = ((long long)(kv->P - 1) * kv->stride_p + (long long)(kv->H_kv - 1) * kv->stride_h) / kv->stride_n + kv->N_max;
    return true;
}

// The prefix cache as a rank-4 tensor: (d, N_max, H_kv, P) with the caller's strides, or (d, page_size, H_kv, num_pages).
inline bool make_cache_map(CUtensorMap *m, const mage_kv_t *kv, const void *base, int eb = 2) {
    const cuuint64_t e = (cuuint64_t)eb;
    if (kv->page_size == 0) {
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)kv->N_max, (cuuint64_t)kv->H_kv, (cuuint64_t)kv->P};
        cuuint64_t str[3] = {(cuuint64_t)kv->stride_n * e, (cuuint64_t)kv->stride_h * e, (cuuint64_t)kv->stride_p * e};
        return make_map(m, base, 4, dims, str, 64, eb);
    }
    cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)kv->page_size, (cuuint64_t)kv->H_kv, (cuuint64_t)kv->num_pages};
    cuuint64_t str[3] = {(cuuint64_t)kD * e, (cuuint64_t)kv->page_size * kD * e, (cuuint64_t)kv->H_kv * kv->page_size * kD * e};
    return make_map(m, base, 4, dims, str, 64, eb);
}

// Key tiles per CTA of the score pass.  One CTA per SM at a time, so the pass lasts about ceil(heads * c / 148)
// rounds of (tiles per CTA + a fixed start cost of about three tile times: the query tile, the row statistics, the
// first key tile); take the number of pieces per head c that minimises that.  Paged pools (sequences of different
// lengths) keep their pieces at most 64 tiles long.
inline int tiles_per_cta_for(long long heads, int N_max, bool paged) {
    const long long tiles_head = (N_max + kTile - 1) / kTile;
    const long long c_max = tiles_head < 148 ? tiles_head : 148;
    long long best_tpc = tiles_head > 0 ? tiles_head : 1;
    double best = 1e300;
    for (long long c = 1; c <= c_max; ++c) {
        const long long tpc = (tiles_head + c - 1) / c;
        if (paged && tpc > 64 && c < c_max) continue;
        const long long rounds = (heads * c + 147) / 148;
        const double cost = (double)rounds * (double)(tpc + 3);
        if (cost < best) { best = cost; best_tpc = tpc; }
    }
    return (int)best_tpc;
}

}  // namespace tc
}  // namespace mage

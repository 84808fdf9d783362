// Quest-style page estimator, per block (the paper's comparison system; Section 2.2 for the estimator, Section 3.1 / Eq. 2
// for its per-block form, Section 5 "Setup" for page size 16 and re-estimation at every step).
//
//   page summaries   kmin[c], kmax[c] = per-channel minimum / maximum of the 16 keys of a page
//   page score       1/(G B) * sum over the block's G*B query rows of  sum_c max(q_c * kmax[c], q_c * kmin[c])
//   selection        the k/16 pages with the largest score; their tokens are the index set of the reuse step
//
// The score is a plain mean over rows of a function that is linear in each of q+ = max(q, 0) and q- = min(q, 0):
//   max(q_c * kmax_c, q_c * kmin_c) = q+_c * kmax_c + q-_c * kmin_c      (kmax_c >= kmin_c)
// so the sum over rows is taken once per KV head (two d-vectors) and a page costs two dot products: the pass reads
// each summary once and is bound by HBM (512 bytes per page).
#pragma once
#include "common.cuh"

namespace mage {
namespace quest {

constexpr int kPage = MAGE_QUEST_PAGE;          // tokens per page
constexpr int kPagesPerCta = 512;               // pages one CTA of the score pass walks

// One warp per (problem, KV head, page): lane l owns channels 4l..4l+3; the 16 rows' loads are all in flight at once.
__global__ void __launch_bounds__(256) build_kernel(KvView kv, int n_pages_max, __nv_bfloat16 *__restrict__ page_min,
                                                    __nv_bfloat16 *__restrict__ page_max, unsigned *status) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const long long total = (long long)kv.P * kv.H_kv * n_pages_max;
    if (warp >= total) return;
    const int page = (int)(warp % n_pages_max);
    const int z = (int)(warp / n_pages_max), p = z / kv.H_kv, h = z % kv.H_kv;
    const int N = seq_len_of(kv, p);
    if (page >= N / kPage) return;              // only whole pages are summarised
    // a page lies inside one cache page (cache pages are multiples of 16 tokens): one table lookup
    const long long off0 = cache_row_offset(kv, p, h, page * kPage, status);
    if (off0 < 0) return;
    const long long row_stride = kv.page_size ? kD : kv.stride_n;
    uint2 v[kPage];
#pragma unroll
    for (int t = 0; t < kPage; ++t) v[t] = *reinterpret_cast<const uint2 *>(kv.k + off0 + t * row_stride + lane * 4);
    __nv_bfloat162 lo0 = *reinterpret_cast<__nv_bfloat162 *>(&v[0].x), lo1 = *reinterpret_cast<__nv_bfloat162 *>(&v[0].y), hi0 = lo0, hi1 = lo1;
#pragma unroll
    for (int t = 1; t < kPage; ++t) {
        const __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&v[t].x), b = *reinterpret_cast<__nv_bfloat162 *>(&v[t].y);
        lo0 = __hmin2(lo0, a); lo1 = __hmin2(lo1, b);
        hi0 = __hmax2(hi0, a); hi1 = __hmax2(hi1, b);
    }
    const size_t o = ((size_t)z * n_pages_max + page) * kD + lane * 4;
    *reinterpret_cast<uint2 *>(page_min + o) = make_uint2(*reinterpret_cast<unsigned *>(&lo0), *reinterpret_cast<unsigned *>(&lo1));
    *reinterpret_cast<uint2 *>(page_max + o) = make_uint2(*reinterpret_cast<unsigned *>(&hi0), *reinterpret_cast<unsigned *>(&hi1));
}

// CTA = (chunk of kPagesPerCta pages, (problem, KV head)).  Prologue: q+ and q- summed over the G*B rows of the head
// (fp32, fixed order) into shared memory; then one warp per page.
__global__ void __launch_bounds__(256) score_kernel(KvView kv, int n_pages_max, const __nv_bfloat16 *__restrict__ q,
                                                    const __nv_bfloat16 *__restrict__ page_min, const __nv_bfloat16 *__restrict__ page_max,
                                                    float *__restrict__ page_scores, int *__restrict__ page_counts) {
    __shared__ float q_pos[kD], q_neg[kD];
    __shared__ float part_pos[16][kD], part_neg[16][kD];
    const int z = blockIdx.y, p = z / kv.H_kv, h = z % kv.H_kv, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_pages = seq_len_of(kv, p) / kPage;
    if (blockIdx.x == 0 && h == 0 && tid == 0) page_counts[p] = n_pages;
    const int page0 = blockIdx.x * kPagesPerCta;
    if (page0 >= n_pages) return;
    {   // thread = (row group t / 16, 16-byte piece t % 16 of a row): rows rg, rg + 16, ... of the head's G*B rows
        const int piece = tid & 15, rg = tid >> 4;
        const __nv_bfloat16 *qh = q + ((long long)(p * kv.H_q + h * kv.G) * kv.B) * kD + piece * 8;
        float sp[8], sn[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) sp[e] = sn[e] = 0.f;
        for (int r = rg; r < kv.M; r += 16) {
            float x[8];
            bf16x8_to_float(*reinterpret_cast<const uint4 *>(qh + (long long)r * kD), x);
#pragma unroll
            for (int e = 0; e < 8; ++e) { sp[e] += fmaxf(x[e], 0.f); sn[e] += fminf(x[e], 0.f); }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) { part_pos[rg][piece * 8 + e] = sp[e]; part_neg[rg][piece * 8 + e] = sn[e]; }
    }
    __syncthreads();
    if (tid < kD) {
        float sp = 0.f, sn = 0.f;
#pragma unroll
        for (int g = 0; g < 16; ++g) { sp += part_pos[g][tid]; sn += part_neg[g][tid]; }     // fixed order
        q_pos[tid] = sp;
        q_neg[tid] = sn;
    }
    __syncthreads();
    const float qp0 = q_pos[lane * 4], qp1 = q_pos[lane * 4 + 1], qp2 = q_pos[lane * 4 + 2], qp3 = q_pos[lane * 4 + 3];
    const float qn0 = q_neg[lane * 4], qn1 = q_neg[lane * 4 + 1], qn2 = q_neg[lane * 4 + 2], qn3 = q_neg[lane * 4 + 3];
    const float inv_m = 1.f / (float)kv.M;
    const int page_end = min(n_pages, page0 + kPagesPerCta);
    // four pages per warp and iteration, their eight loads issued before any is used
    for (int pg0 = page0 + warp; pg0 < page_end; pg0 += 32) {
        uint2 a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int pg = pg0 + 8 * u;
            if (pg < page_end) {
                const size_t o = ((size_t)z * n_pages_max + pg) * kD + lane * 4;
                a[u] = *reinterpret_cast<const uint2 *>(page_max + o);
                b[u] = *reinterpret_cast<const uint2 *>(page_min + o);
            } else {
                a[u] = b[u] = make_uint2(0u, 0u);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int pg = pg0 + 8 * u;
            const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a[u].x)), a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a[u].y));
            const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b[u].x)), b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b[u].y));
            float s = qp0 * a0.x + qn0 * b0.x;
            s = fmaf(qp1, a0.y, fmaf(qn1, b0.y, s));
            s = fmaf(qp2, a1.x, fmaf(qn2, b1.x, s));
            s = fmaf(qp3, a1.y, fmaf(qn3, b1.y, s));
#pragma unroll
            for (int w = 16; w; w >>= 1) s += __shfl_xor_sync(0xffffffffu, s, w);
            if (lane == 0 && pg < page_end) page_scores[(size_t)z * n_pages_max + pg] = s * inv_m;
        }
    }
}

// CTA = (problem, KV head): the selected pages (ascending, as the page top-k wrote them) become token positions.
__global__ void __launch_bounds__(256) expand_kernel(int H_kv, int k, const int *__restrict__ page_idx, const int *__restrict__ pages_sel,
                                                     int *__restrict__ indices, int *__restrict__ k_eff) {
    const int z = blockIdx.x, p = z / H_kv, h = z % H_kv, k_pages = k / kPage;
    const int n_sel = min(max(pages_sel[p], 0), k_pages);
    const int *src = page_idx + (size_t)z * k_pages;
    int *dst = indices + (size_t)z * k;
    for (int t = threadIdx.x; t < k; t += blockDim.x) {
        const int i = t / kPage;
        dst[t] = i < n_sel ? src[i] * kPage + (t % kPage) : -1;
    }
    if (h == 0 && threadIdx.x == 0) k_eff[p] = n_sel * kPage;
}

}  // namespace quest
}  // namespace mage

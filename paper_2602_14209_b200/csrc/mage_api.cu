// Host side of libmage: argument validation, workspace planning and kernel launches behind the C ABI.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <mutex>

#include "common.cuh"
#include "k8.cuh"
#include "prune.cuh"
#include "quest.cuh"
#include "simt_kernels.cuh"
#include "tc_host.cuh"
#include "topk.cuh"

namespace mage {

static std::atomic<uint64_t> g_launches{0};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool valid_kv(const mage_kv_t *kv, mage_status *why) {
    auto fail = [&](mage_status s) { if (why) *why = s; return false; };
    if (!kv) return fail(MAGE_ERR_INVALID_ARG);
    if (kv->P < 1 || kv->H_q < 1 || kv->H_kv < 1 || kv->H_q % kv->H_kv != 0 || kv->B < 1 || kv->N_max < 0 || kv->d < 1)
        return fail(MAGE_ERR_INVALID_ARG);
    if (kv->d != kD || kv->B > 64) return fail(MAGE_ERR_UNSUPPORTED);
    if (kv->N_max > 0 && (!kv->k_cache || !kv->v_cache)) return fail(MAGE_ERR_INVALID_ARG);
    if (kv->page_size < 0) return fail(MAGE_ERR_INVALID_ARG);
    if (kv->page_size == 0) {
        if (kv->stride_n < kD || kv->stride_n % 8 || kv->stride_h % 8 || kv->stride_p % 8 || kv->stride_h < 0 || kv->stride_p < 0)
            return fail(MAGE_ERR_INVALID_ARG);
    } else {
        if (kv->page_size < 16 || (kv->page_size & (kv->page_size - 1))) return fail(MAGE_ERR_UNSUPPORTED);
        if (kv->N_max > 0 && (!kv->block_table || kv->num_pages < 1)) return fail(MAGE_ERR_INVALID_ARG);
        if ((int64_t)kv->max_pages * kv->page_size < kv->N_max) return fail(MAGE_ERR_INVALID_ARG);
    }
    if ((int64_t)kv->P * kv->H_kv > 65535) return fail(MAGE_ERR_UNSUPPORTED);      // (problem, KV head) pairs are one grid dimension
    return true;
}

static KvView make_view(const mage_kv_t *kv) {
    KvView v;
    v.k = static_cast<const __nv_bfloat16 *>(kv->k_cache);
    v.v = static_cast<const __nv_bfloat16 *>(kv->v_cache);
    v.stride_p = kv->stride_p; v.stride_h = kv->stride_h; v.stride_n = kv->stride_n;
    v.block_table = kv->block_table; v.seq_lens = kv->seq_lens;
    v.max_pages = kv->max_pages; v.num_pages = kv->num_pages; v.page_size = kv->page_size;
    v.N_max = kv->N_max;
    v.P = kv->P; v.H_q = kv->H_q; v.H_kv = kv->H_kv; v.B = kv->B; v.G = kv->H_q / kv->H_kv; v.M = v.G * kv->B;
    return v;
}

// Split of the prefix for the exact pass into chunks of whole 128-key tiles.  Large jobs get about 12 waves of CTAs
// over the 148 SMs (good balance, partial results stay a few percent of the K/V traffic); small jobs get one wave
// with at least ~32 tiles per CTA, because every extra chunk costs a CTA prologue and a row in the merge.
// Pure function of the description.
static Plan make_plan(const mage_kv_t *kv, int k_max = 0) {
    Plan pl;
    pl.M = kv->H_q / kv->H_kv * kv->B;
    pl.Mw = (int)align_up(pl.M, 128);
    const int64_t heads = (int64_t)kv->P * kv->H_kv;
    const int64_t tiles_head = kv->N_max > 0 ? (kv->N_max + 127) / 128 : 1;
    // Key chunks per head.  One CTA per (head, chunk) and one CTA per SM at a time, so the pass lasts
    // about ceil(heads * c / 148) rounds of (tiles per chunk + a fixed start/finish cost of about four tile times); each
    // chunk also costs a partial result written and merged.  Pick the c that minimises that estimate.  A paged pool
    // usually holds sequences of different lengths, which N_max says nothing about: keep its chunks at most 64 tiles
    // long so that the long sequences spread over many CTAs.
    int64_t want = 1;
    double best = 1e300;
    const int64_t c_max = tiles_head < 148 ? tiles_head : 148;
    for (int64_t c = 1; c <= c_max; ++c) {
        const int64_t tiles_c = (tiles_head + c - 1) / c;
        if (kv->page_size != 0 && tiles_c > 64 && c < c_max) continue;
        // (the CTA for the block's own keys costs about five tile times and takes an SM like any other)
        const double per_cta = (double)(tiles_c + 4), work = (double)(heads * c) * per_cta + 5.0 * (double)heads;
        const double rounds = std::ceil(work / (148.0 * per_cta) - 1e-9);
        const double cost = rounds * per_cta + 7.7e-5 * (double)heads * pl.M * (double)c;
        if (cost < best) { best = cost; want = c; }
    }
    int64_t len = kv->N_max > 0 ? (kv->N_max + want - 1) / want : 128;
    len = (int64_t)align_up((size_t)len, 128);
    pl.chunk_len = (int)len;
    pl.n_chunks = kv->N_max > 0 ? (int)((kv->N_max + len - 1) / len) : 0;
    const size_t items = (size_t)heads * (pl.n_chunks + 1);
    size_t off = 0;
    pl.off_part_o = off;  off += items * pl.Mw * kD;
    pl.off_part_ml = off; off += items * pl.Mw * 2;
    pl.off_neg_lse = off; off += (size_t)heads * pl.Mw;
    pl.exact_bytes = align_up(off * sizeof(float), 256);
    // reuse step: when a launch has few (head, row-group) pairs, the selected keys of one head are split over several
    // CTAs whose partial results are merged by a second small kernel; room for that, sized by the largest budget
    off = pl.exact_bytes / sizeof(float);
    const int tiles_max = k_max > 0 ? (k_max + kv->B + 127) / 128 : 0;
    pl.sparse_split_max = tiles_max < 32 ? tiles_max : 32;
    pl.off_sparse_o = off;  off += (size_t)heads * pl.sparse_split_max * pl.Mw * kD;
    pl.off_sparse_ml = off; off += (size_t)heads * pl.sparse_split_max * pl.Mw * 2;
    pl.total_bytes = align_up(off * sizeof(float), 256);
    return pl;
}

// Launch with the programmatic-serialization attribute: the kernel may be scheduled while its predecessor in the stream is
// still running; every kernel launched this way begins with griddepcontrol.wait, so it touches no global memory before
// the predecessor has completed.  What is saved is the launch gap between dependent kernels (a few microseconds each,
// which is most of a single-layer reuse step).
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

static mage_status launch_check() {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        std::fprintf(stderr, "libmage: kernel launch failed: %s\n", cudaGetErrorString(e));
        return MAGE_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return MAGE_OK;
}

// Raise a kernel's dynamic shared memory limit; done once per kernel and device, remembered afterwards.
static mage_status opt_in_smem_impl(const void *kernel, size_t bytes) {
    static std::mutex mu;
    static const void *seen[32];
    static unsigned long long seen_devs[32];
    static int n_seen = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MAGE_ERR_CUDA;
    const unsigned long long bit = 1ull << (dev & 63);
    std::lock_guard<std::mutex> lock(mu);
    int slot = -1;
    for (int i = 0; i < n_seen; ++i)
        if (seen[i] == kernel) slot = i;
    if (slot >= 0 && (seen_devs[slot] & bit)) return MAGE_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return MAGE_ERR_CUDA;
    if (slot < 0 && n_seen < 32) { slot = n_seen++; seen[slot] = kernel; seen_devs[slot] = 0; }
    if (slot >= 0) seen_devs[slot] |= bit;
    return MAGE_OK;
}
template <typename K>
static mage_status opt_in_smem(K kernel, size_t bytes) { return opt_in_smem_impl(reinterpret_cast<const void *>(kernel), bytes); }

// Why the tensor-core kernels cannot take this description, or MAGE_OK.  There is one production path; the portable
// CUDA-core kernels run only when the caller asks for them with MAGE_FLAG_SIMT_KERNELS, never as a silent substitute.
static mage_status tc_supported(const mage_kv_t *kv) {   // (8-bit keys: the caller's copy of kv carries the codes as k_cache)
    if (kv->page_size != 0 && kv->page_size % 64 != 0) return MAGE_ERR_UNSUPPORTED;        // a 64-key TMA box must lie inside one page
    if (kv->N_max > 0 && ((reinterpret_cast<uintptr_t>(kv->k_cache) | reinterpret_cast<uintptr_t>(kv->v_cache)) & 15)) return MAGE_ERR_UNSUPPORTED;
    if (tc::encode_fn() == nullptr) return MAGE_ERR_CUDA;
    return MAGE_OK;
}

// The block-score pass (Eq. 4) over all key tiles, or over the tiles of `list`: grid_x CTAs of tiles_per_cta tiles per head.
static mage_status launch_score_pass(const KvView &view, const Plan &plan, const CUtensorMap &map_q_rows, const CUtensorMap &map_k,
                                     int grid_x, int tiles_per_cta, float scale_log2, const float *ws, float *scores,
                                     unsigned *dev_status, cudaStream_t st, const tc::ScoreTileList &list,
                                     const float *qk_scale = nullptr) {
    dim3 sgrid(grid_x, view.P * view.H_kv, 1);
    for (int r0 = 0; r0 < view.M; r0 += 256) {
        launch_pdl(qk_scale ? tc::score_kernel<true> : tc::score_kernel<false>, sgrid, dim3(tc::kScoreThreads), tc::kScoreSmemBytes, st, map_q_rows, map_k, view, plan, r0, std::min(256, view.M - r0),
                   tiles_per_cta, scale_log2, ws, scores, (int)(r0 > 0), dev_status, list, qk_scale);
        if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    }
    return MAGE_OK;
}

// Step 1 (Algorithm 1, Phase 1): the exact pass over prefix + block keys, the merge of its per-chunk partial results and
// the block-score pass.  scores_only: the select stream's own computation (Algorithm 1: A = softmax(Q K^T / sqrt d) over
// the prefix, then the mean over the block's rows) without the attention output: pass A keeps only the rows' maxima and
// sums (no V, no P V, no block keys), the merge emits only the log-sum-exp, pass B is unchanged; k_blk, v_blk, out unused.
// 8-bit keys: the codes of the cache with their scales (caller's), and the per-call scratch of the codes of the queries and
// the block's keys with the heads' factors s_q s_k.
struct K8 {
    const uint8_t *k8;
    const float *k_scale;
    uint8_t *q8, *kb8;
    float *qk_scale;
};
static size_t k8_scratch_layout(const mage_kv_t *kv, size_t *off_kb8, size_t *off_qk) {
    const size_t q8 = align_up((size_t)kv->P * kv->H_q * kv->B * kD, 256), kb8 = align_up((size_t)kv->P * kv->H_kv * kv->B * kD, 256);
    if (off_kb8) *off_kb8 = q8;
    if (off_qk) *off_qk = q8 + kb8;
    return q8 + kb8 + align_up((size_t)kv->P * kv->H_kv * sizeof(float), 256);
}
// Codes of the call's queries and block keys (one small kernel in front of the pass that uses them).
static mage_status launch_block_codes(const KvView &view, const K8 &k8, const __nv_bfloat16 *q, const __nv_bfloat16 *k_blk, cudaStream_t st) {
    launch_pdl(k8::block_code_kernel, dim3(view.P * view.H_kv), dim3(256), 0, st, view, q, k_blk, k8.k_scale, k8.q8, k8.kb8, k8.qk_scale);
    return launch_check();
}

static mage_status launch_exact_select(const mage_kv_t *kv, const KvView &view, const Plan &plan, const __nv_bfloat16 *q,
                                       const __nv_bfloat16 *k_blk, const __nv_bfloat16 *v_blk, float sm_scale,
                                       __nv_bfloat16 *out, float *scores, float *ws, unsigned *dev_status, cudaStream_t st,
                                       cudaEvent_t *ev, bool scores_only = false, float2 *rowsum = nullptr, int rowsum_tiles = 0,
                                       const K8 *k8 = nullptr) {
    const float scale_log2 = sm_scale * kLog2e;
    const int heads = kv->P * kv->H_kv, rows_total = heads * view.M;
    const int n_items = plan.n_chunks + (scores_only ? 0 : 1);
    if (k8 && ((kv->flags & MAGE_FLAG_SIMT_KERNELS) || scores_only)) return MAGE_ERR_UNSUPPORTED;
    if (kv->flags & MAGE_FLAG_SIMT_KERNELS) {
        using namespace simt;
        auto kern = attn_kernel<Mode::kExactPartial>;
        if (opt_in_smem(kern, kSmemBytes) != MAGE_OK || opt_in_smem(simt::score_kernel, kSmemBytes) != MAGE_OK) return MAGE_ERR_CUDA;
        if (ev) cudaEventRecord(ev[0], st);
        if (n_items > 0) {
            kern<<<dim3((view.M + kRows - 1) / kRows, n_items, heads), kThreads, kSmemBytes, st>>>(view, plan, q, k_blk, v_blk, nullptr, nullptr, 0, scale_log2, ws, nullptr, dev_status);
            if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
        }
        if (ev) cudaEventRecord(ev[1], st);
        launch_pdl(combine_kernel, dim3((rows_total + 3) / 4), dim3(128), 0, st, view, plan, ws, out, (int)scores_only);
        if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
        if (ev) cudaEventRecord(ev[2], st);
        if (scores && kv->N_max > 0) {
            simt::score_kernel<<<dim3((kv->N_max + kKeys - 1) / kKeys, 1, heads), kThreads, kSmemBytes, st>>>(view, plan, q, scale_log2, ws, scores, dev_status);
            if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
        }
        if (ev) cudaEventRecord(ev[3], st);
        return MAGE_OK;
    }
    const mage_status sup = tc_supported(kv);
    if (sup != MAGE_OK) return sup;
    // every tensor map is encoded before the first launch: a description that cannot be encoded launches nothing
    tc::AttnMaps maps;
    CUtensorMap map_q_rows, map_k_score;
    auto kern_tc = k8 ? tc::attn_kernel<false, true> : tc::attn_kernel<false, false>;
    const int eb = k8 ? 1 : 2;                             // bytes per query / key element
    const void *q_src = k8 ? (const void *)k8->q8 : (const void *)q, *kc_src = k8 ? (const void *)k8->k8 : kv->k_cache;
    const void *kb_src = k8 ? (const void *)k8->kb8 : (const void *)k_blk;
    bool maps_ok = tc::make_group_rows_map(&maps.q, q_src, heads, view.M, eb);
    if (maps_ok && kv->N_max > 0) maps_ok = tc::make_cache_map(&maps.k, kv, kc_src, eb);
    else maps.k = maps.q;                                  // no prefix: never used
    if (k8) maps.qk_scale = k8->qk_scale;
    if (maps_ok && scores_only) {
        maps.v = maps.kb = maps.vb = maps.k;              // never used in this mode
        maps.lse_only = 1;
    } else if (maps_ok) {
        maps_ok = tc::make_rows_map(&maps.kb, kb_src, (long long)heads * kv->B, eb) && tc::make_rows_map(&maps.vb, v_blk, (long long)heads * kv->B);
        if (maps_ok && kv->N_max > 0) maps_ok = tc::make_cache_map(&maps.v, kv, kv->v_cache);
        else maps.v = maps.q;
    }
    maps.test_stall = (kv->flags & MAGE_FLAG_TEST_STALL) ? 1 : 0;
    maps.rowsum = rowsum;
    maps.rowsum_tiles = rowsum_tiles;
    const bool want_scores = scores && kv->N_max > 0;
    if (maps_ok && want_scores) maps_ok = tc::make_rows_map(&map_q_rows, q_src, (long long)kv->P * kv->H_q * kv->B, eb) && tc::make_cache_map(&map_k_score, kv, kc_src, eb);
    if (!maps_ok) return MAGE_ERR_UNSUPPORTED;
    if (opt_in_smem(kern_tc, tc::kAttnSmemBytesDense) != MAGE_OK || opt_in_smem(tc::score_kernel<false>, tc::kScoreSmemBytes) != MAGE_OK ||
        opt_in_smem(tc::score_kernel<true>, tc::kScoreSmemBytes) != MAGE_OK)
        return MAGE_ERR_CUDA;
    if (ev) cudaEventRecord(ev[0], st);
    if (k8 && launch_block_codes(view, *k8, q, k_blk, st) != MAGE_OK) return MAGE_ERR_CUDA;
    if (n_items > 0) {
        launch_pdl(kern_tc, dim3(n_items, (view.M + 255) / 256, heads), dim3(320), tc::kAttnSmemBytesDense, st, maps, view, plan, k_blk, v_blk, (const int *)nullptr,
                   (const int *)nullptr, 0, scale_log2, ws, (__nv_bfloat16 *)nullptr, dev_status);
        if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    }
    if (ev) cudaEventRecord(ev[1], st);
    launch_pdl(combine_kernel, dim3((rows_total + 3) / 4), dim3(128), 0, st, view, plan, ws, out, (int)scores_only);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    if (ev) cudaEventRecord(ev[2], st);
    if (want_scores) {
        const int tpc = tc::tiles_per_cta_for(heads, kv->N_max, kv->page_size != 0);
        const int tiles_head = (kv->N_max + tc::kTile - 1) / tc::kTile;
        if (launch_score_pass(view, plan, map_q_rows, map_k_score, (tiles_head + tpc - 1) / tpc, tpc, scale_log2, ws, scores, dev_status, st, tc::ScoreTileList(),
                              k8 ? k8->qk_scale : nullptr) != MAGE_OK)
            return MAGE_ERR_CUDA;
    }
    if (ev) cudaEventRecord(ev[3], st);
    return MAGE_OK;
}

// Reuse step (Algorithm 1, Phase 2).
static mage_status launch_sparse_step(const mage_kv_t *kv, const KvView &view, const Plan &plan, const __nv_bfloat16 *q,
                                      const __nv_bfloat16 *k_blk, const __nv_bfloat16 *v_blk, const int *indices,
                                      const int *k_eff, int k, float sm_scale, __nv_bfloat16 *out, float *ws, bool ws_ok,
                                      unsigned *dev_status, cudaStream_t st, const K8 *k8 = nullptr) {
    const int heads = kv->P * kv->H_kv;
    if (k8 && (kv->flags & MAGE_FLAG_SIMT_KERNELS)) return MAGE_ERR_UNSUPPORTED;
    if (kv->flags & MAGE_FLAG_SIMT_KERNELS) {
        using namespace simt;
        auto kern = attn_kernel<Mode::kSparseFinal>;
        if (opt_in_smem(kern, kSmemBytes) != MAGE_OK) return MAGE_ERR_CUDA;
        kern<<<dim3((view.M + kRows - 1) / kRows, 1, heads), kThreads, kSmemBytes, st>>>(view, plan, q, k_blk, v_blk, indices, k_eff, k, sm_scale * kLog2e, nullptr, out, dev_status);
        return launch_check();
    }
    if (tc::encode_fn() == nullptr) return MAGE_ERR_CUDA;
    tc::AttnMaps maps;
    auto kern_tc = k8 ? tc::attn_kernel<true, true> : tc::attn_kernel<true, false>;
    const int eb = k8 ? 1 : 2;
    const void *q_src = k8 ? (const void *)k8->q8 : (const void *)q, *kc_src = k8 ? (const void *)k8->k8 : kv->k_cache;
    const void *kb_src = k8 ? (const void *)k8->kb8 : (const void *)k_blk;
    if (!tc::make_group_rows_map(&maps.q, q_src, heads, view.M, eb)) return MAGE_ERR_UNSUPPORTED;
    // 8-bit keys with one row group per head: the kernel codes the queries and the block's keys itself (no kernel in front)
    const bool k8_fused = k8 && view.M <= 256;
    if (k8) maps.qk_scale = k8->qk_scale;
    if (k8_fused) {
        maps.q_raw = q;
        maps.k_scale = k8->k_scale;
    }
    maps.k = maps.v = maps.kb = maps.vb = maps.q;         // placeholders unless the TMA row gather below applies
    // Two gathers inside the one kernel: single 256-byte rows by TMA when the cache is one list of rows with a single pitch
    // (every paged pool; contiguous layouts whose head and problem strides are multiples of the row stride), otherwise
    // 16-byte cp.async, which addresses rows through 32-bit offsets in 16-byte units.
    long long c_rows = 0, c_pitch = 0;
    const long long b_rows = (long long)heads * kv->B;
    const bool aligned = !((reinterpret_cast<uintptr_t>(kc_src) | reinterpret_cast<uintptr_t>(kv->v_cache) | reinterpret_cast<uintptr_t>(kb_src) |
                            reinterpret_cast<uintptr_t>(v_blk)) & 15);
    if (kv->N_max > 0 && aligned && tc::cache_as_rows(kv, &c_rows, &c_pitch) && tc::make_row_gather_map(&maps.k, kc_src, c_rows, c_pitch, eb) &&
        tc::make_row_gather_map(&maps.v, kv->v_cache, c_rows, c_pitch) && tc::make_row_gather_map(&maps.kb, kb_src, b_rows, kD, eb) &&
        tc::make_row_gather_map(&maps.vb, v_blk, b_rows, kD)) {
        maps.gather_rows = (int)c_rows;
        maps.gather_blk_rows = (int)b_rows;
        maps.gather_pitch = (int)c_pitch;
    } else if (k8) {                                       // 8-bit keys are gathered by TMA only (a cache with one row pitch)
        if (kv->N_max != 0 || !aligned || !tc::make_row_gather_map(&maps.kb, kb_src, b_rows, kD, eb) || !tc::make_row_gather_map(&maps.vb, v_blk, b_rows, kD))
            return MAGE_ERR_UNSUPPORTED;
        maps.k = maps.kb;                                  // no prefix: every request names the block's rows
        maps.v = maps.vb;
        maps.gather_rows = maps.gather_blk_rows = (int)b_rows;
        maps.gather_pitch = kD;
    } else {
        if (!aligned) return MAGE_ERR_UNSUPPORTED;        // cp.async moves 16-byte pieces
        const long long last = kv->page_size ? (long long)kv->num_pages * kv->H_kv * kv->page_size * kD
                                             : (long long)(kv->P - 1) * kv->stride_p + (long long)(kv->H_kv - 1) * kv->stride_h + (long long)kv->N_max * kv->stride_n;
        if ((last >> 3) > 0x7fffffffLL) return MAGE_ERR_UNSUPPORTED;
    }
    if (opt_in_smem(kern_tc, tc::kAttnSmemBytesSparse) != MAGE_OK) return MAGE_ERR_CUDA;
    int n_rg = (view.M + 255) / 256;
    // few (head, row-group) pairs in the launch: split each head's keys over several CTAs and merge
    int n_split = 1;
    if (ws_ok && plan.sparse_split_max > 1) {
        const int tiles = (k + kv->B + 127) / 128;
        auto splits_for = [&](int groups) {
            int s = 148 / (heads * groups);
            if (s > tiles) s = tiles;
            if (s > plan.sparse_split_max) s = plan.sparse_split_max;
            return s < 1 ? 1 : s;
        };
        n_split = splits_for(n_rg);
        // A split CTA spends most of its time writing its partial result (fp32, 512 bytes per query row); with row groups of
        // 128 instead of 256 rows each CTA writes half of it.  Every key tile is then gathered by two CTAs, which costs more
        // than it saves once the launch fills more than about half of the SMs (measured: 12.9 -> 11.4 us with 40 CTAs,
        // 15.8 -> 17.3 us with 136).
        const int n_rg128 = (view.M + 127) / 128;
        if (n_split > 1 && n_rg128 > n_rg && !k8_fused && splits_for(n_rg128) == n_split && heads * n_rg128 * n_split <= 74) {
            n_rg = n_rg128;
            maps.rg_rows = 128;
        }
    }
    if (k8 && !k8_fused && launch_block_codes(view, *k8, q, k_blk, st) != MAGE_OK) return MAGE_ERR_CUDA;
    launch_pdl(kern_tc, dim3(n_split, n_rg, heads), dim3(tc::kSparseThreads), tc::kAttnSmemBytesSparse, st, maps, view, plan, k_blk, v_blk, indices, k_eff, k, sm_scale * kLog2e, ws, out, dev_status);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    if (n_split > 1) {
        launch_pdl(tc::sparse_combine_kernel, dim3((heads * view.M + 3) / 4), dim3(128), 0, st, view, plan, n_split, k, k_eff, (const float *)ws, out);
        return launch_check();
    }
    return MAGE_OK;
}

}  // namespace mage

using namespace mage;

extern "C" {

size_t mage_workspace_bytes(const mage_kv_t *kv, int32_t k_max) {
    if (!valid_kv(kv, nullptr) || k_max < 1) return 0;
    return make_plan(kv, k_max).total_bytes;
}

mage_status mage_exact_select_events(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                                     float sm_scale, void *out, float *scores, void *workspace, size_t workspace_bytes,
                                     uint32_t *dev_status, void *stream, void **events) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!q || !k_blk || !v_blk || !out || !workspace || (kv->N_max > 0 && !scores)) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f) || (reinterpret_cast<uintptr_t>(workspace) & 255)) return MAGE_ERR_INVALID_ARG;
    const Plan plan = make_plan(kv);
    if (workspace_bytes < plan.exact_bytes) return MAGE_ERR_WORKSPACE;
    const KvView view = make_view(kv);
    return launch_exact_select(kv, view, plan, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_blk),
                             static_cast<const __nv_bfloat16 *>(v_blk), sm_scale, static_cast<__nv_bfloat16 *>(out), scores,
                             static_cast<float *>(workspace), dev_status, static_cast<cudaStream_t>(stream),
                             reinterpret_cast<cudaEvent_t *>(events));
}

mage_status mage_exact_select(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk, float sm_scale,
                              void *out, float *scores, void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                              void *stream) {
    return mage_exact_select_events(kv, q, k_blk, v_blk, sm_scale, out, scores, workspace, workspace_bytes, dev_status,
                                    stream, nullptr);
}

mage_status mage_exact_attn(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk, float sm_scale,
                            void *out, void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!q || !k_blk || !v_blk || !out || !workspace) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f) || (reinterpret_cast<uintptr_t>(workspace) & 255)) return MAGE_ERR_INVALID_ARG;
    const Plan plan = make_plan(kv);
    if (workspace_bytes < plan.exact_bytes) return MAGE_ERR_WORKSPACE;
    const KvView view = make_view(kv);
    return launch_exact_select(kv, view, plan, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_blk),
                             static_cast<const __nv_bfloat16 *>(v_blk), sm_scale, static_cast<__nv_bfloat16 *>(out), nullptr,
                             static_cast<float *>(workspace), dev_status, static_cast<cudaStream_t>(stream), nullptr);
}

mage_status mage_select_scores(const mage_kv_t *kv, const void *q, float sm_scale, float *scores, void *workspace,
                               size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!q || !workspace || (kv->N_max > 0 && !scores)) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f) || (reinterpret_cast<uintptr_t>(workspace) & 255)) return MAGE_ERR_INVALID_ARG;
    const Plan plan = make_plan(kv);
    if (workspace_bytes < plan.exact_bytes) return MAGE_ERR_WORKSPACE;
    if (kv->N_max == 0) return MAGE_OK;                   // no prefix: no score to write
    const KvView view = make_view(kv);
    return launch_exact_select(kv, view, plan, static_cast<const __nv_bfloat16 *>(q), nullptr, nullptr, sm_scale, nullptr, scores,
                             static_cast<float *>(workspace), dev_status, static_cast<cudaStream_t>(stream), nullptr, true);
}

mage_status mage_topk(const float *scores, const int32_t *seq_lens, int32_t P, int32_t H_kv, int32_t N_max, int32_t k,
                      int32_t *indices, int32_t *k_eff, void *workspace, size_t workspace_bytes, void *stream) {
    (void)workspace; (void)workspace_bytes;
    if (P < 1 || H_kv < 1 || N_max < 0 || k < 1 || !indices || !k_eff || (N_max > 0 && !scores)) return MAGE_ERR_INVALID_ARG;
    // long rows of a few heads: a cluster of eight CTAs per head shares the row; otherwise one CTA per head
    // (few heads only: a cluster member costs a whole SM for about 25 us whatever the row length, so with many heads the
    // single-CTA kernel, one SM per head, finishes sooner)
    if (N_max >= 16384 && P * H_kv * kTopkCluster <= 148) {
        if (opt_in_smem(topk_cluster_kernel, kTopkClusterSmem) != MAGE_OK) return MAGE_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kTopkCluster, P * H_kv, 1);
        cfg.blockDim = dim3(kTopkThreads);
        cfg.dynamicSmemBytes = kTopkClusterSmem;
        cfg.stream = static_cast<cudaStream_t>(stream);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kTopkCluster;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaLaunchKernelEx(&cfg, topk_cluster_kernel, scores, seq_lens, H_kv, N_max, k, indices, k_eff);
        return launch_check();
    }
    topk_kernel<<<P * H_kv, kTopkThreads, 0, static_cast<cudaStream_t>(stream)>>>(scores, seq_lens, H_kv, N_max, k, indices, k_eff);
    return launch_check();
}

mage_status mage_sparse_block_attn(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                                   const int32_t *indices, const int32_t *k_eff, int32_t k, float sm_scale, void *out,
                                   void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!q || !k_blk || !v_blk || !out || !indices || !k_eff || k < 1) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f)) return MAGE_ERR_INVALID_ARG;
    const Plan plan = make_plan(kv, k);
    const KvView view = make_view(kv);
    const bool ws_ok = workspace && !(reinterpret_cast<uintptr_t>(workspace) & 255) && workspace_bytes >= plan.total_bytes;
    return launch_sparse_step(kv, view, plan, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_blk),
                       static_cast<const __nv_bfloat16 *>(v_blk), indices, k_eff, k, sm_scale, static_cast<__nv_bfloat16 *>(out),
                       static_cast<float *>(workspace), ws_ok, dev_status, static_cast<cudaStream_t>(stream));
}

// ---- 8-bit keys
static bool valid_k8(const mage_kv_t *kv, const mage_k8_t *k8, K8 *out) {
    if (!k8 || !k8->scratch || (reinterpret_cast<uintptr_t>(k8->scratch) & 255)) return false;
    if (kv->N_max > 0 && (!k8->k8_cache || !k8->k_scale)) return false;
    if (!k8->k_scale) return false;
    size_t off_kb8 = 0, off_qk = 0;
    k8_scratch_layout(kv, &off_kb8, &off_qk);
    uint8_t *base = static_cast<uint8_t *>(k8->scratch);
    out->k8 = static_cast<const uint8_t *>(k8->k8_cache);
    out->k_scale = k8->k_scale;
    out->q8 = base;
    out->kb8 = base + off_kb8;
    out->qk_scale = reinterpret_cast<float *>(base + off_qk);
    return true;
}

size_t mage_k8_scratch_bytes(const mage_kv_t *kv) {
    if (!valid_kv(kv, nullptr)) return 0;
    return k8_scratch_layout(kv, nullptr, nullptr);
}

mage_status mage_k8_quantize_cache(const mage_kv_t *kv, int32_t row_begin, void *k8_cache, float *k_scale, uint32_t *dev_status, void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!k_scale || row_begin < 0 || (kv->N_max > 0 && !k8_cache)) return MAGE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(k8_cache) | reinterpret_cast<uintptr_t>(kv->k_cache)) & 15) return MAGE_ERR_UNSUPPORTED;
    if (kv->page_size == 0 && (kv->stride_n % 16 || kv->stride_h % 16 || kv->stride_p % 16)) return MAGE_ERR_UNSUPPORTED;   // 16 codes per store
    const KvView view = make_view(kv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int heads = kv->P * kv->H_kv;
    const int rows = kv->N_max - row_begin;
    if (row_begin == 0) {                                  // the scales are taken from the rows that are there now
        if (cudaMemsetAsync(k_scale, 0, (size_t)heads * sizeof(float), st) != cudaSuccess) return MAGE_ERR_CUDA;
        if (rows > 0) {
            k8::cache_amax_kernel<<<dim3((rows + k8::kRowsPerCta - 1) / k8::kRowsPerCta, heads), 256, 0, st>>>(view, 0, reinterpret_cast<unsigned *>(k_scale), dev_status);
            if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
        }
        k8::amax_to_scale_kernel<<<(heads + 127) / 128, 128, 0, st>>>(k_scale, heads);
        if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    }
    if (rows > 0) {
        k8::cache_code_kernel<<<dim3((rows + k8::kRowsPerCta - 1) / k8::kRowsPerCta, heads), 256, 0, st>>>(view, row_begin, k_scale, static_cast<uint8_t *>(k8_cache), dev_status);
        if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    }
    return MAGE_OK;
}

mage_status mage_exact_select_k8_events(const mage_kv_t *kv, const mage_k8_t *k8, const void *q, const void *k_blk, const void *v_blk,
                                        float sm_scale, void *out, float *scores, void *workspace, size_t workspace_bytes,
                                        uint32_t *dev_status, void *stream, void **events) {
    if (!kv || !k8) return MAGE_ERR_INVALID_ARG;
    mage_kv_t kvc = *kv;
    kvc.k_cache = k8->k8_cache;                            // the 16-bit keys are not read
    mage_status why = MAGE_OK;
    if (!valid_kv(&kvc, &why)) return why;
    K8 a;
    if (!valid_k8(&kvc, k8, &a)) return MAGE_ERR_INVALID_ARG;
    if (!q || !k_blk || !v_blk || !out || !workspace || (kvc.N_max > 0 && !scores)) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f) || (reinterpret_cast<uintptr_t>(workspace) & 255)) return MAGE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_blk)) & 15) return MAGE_ERR_UNSUPPORTED;
    const Plan plan = make_plan(&kvc);
    if (workspace_bytes < plan.exact_bytes) return MAGE_ERR_WORKSPACE;
    const KvView view = make_view(&kvc);
    return launch_exact_select(&kvc, view, plan, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_blk),
                               static_cast<const __nv_bfloat16 *>(v_blk), sm_scale, static_cast<__nv_bfloat16 *>(out), scores,
                               static_cast<float *>(workspace), dev_status, static_cast<cudaStream_t>(stream),
                               reinterpret_cast<cudaEvent_t *>(events), false, nullptr, 0, &a);
}

mage_status mage_exact_select_k8(const mage_kv_t *kv, const mage_k8_t *k8, const void *q, const void *k_blk, const void *v_blk,
                                 float sm_scale, void *out, float *scores, void *workspace, size_t workspace_bytes,
                                 uint32_t *dev_status, void *stream) {
    return mage_exact_select_k8_events(kv, k8, q, k_blk, v_blk, sm_scale, out, scores, workspace, workspace_bytes, dev_status, stream, nullptr);
}

mage_status mage_sparse_block_attn_k8(const mage_kv_t *kv, const mage_k8_t *k8, const void *q, const void *k_blk, const void *v_blk,
                                      const int32_t *indices, const int32_t *k_eff, int32_t k, float sm_scale, void *out,
                                      void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream) {
    if (!kv || !k8) return MAGE_ERR_INVALID_ARG;
    mage_kv_t kvc = *kv;
    kvc.k_cache = k8->k8_cache;
    mage_status why = MAGE_OK;
    if (!valid_kv(&kvc, &why)) return why;
    K8 a;
    if (!valid_k8(&kvc, k8, &a)) return MAGE_ERR_INVALID_ARG;
    if (!q || !k_blk || !v_blk || !out || !indices || !k_eff || k < 1) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f)) return MAGE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_blk)) & 15) return MAGE_ERR_UNSUPPORTED;
    const Plan plan = make_plan(&kvc, k);
    const KvView view = make_view(&kvc);
    const bool ws_ok = workspace && !(reinterpret_cast<uintptr_t>(workspace) & 255) && workspace_bytes >= plan.total_bytes;
    return launch_sparse_step(&kvc, view, plan, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_blk),
                              static_cast<const __nv_bfloat16 *>(v_blk), indices, k_eff, k, sm_scale, static_cast<__nv_bfloat16 *>(out),
                              static_cast<float *>(workspace), ws_ok, dev_status, static_cast<cudaStream_t>(stream), &a);
}

mage_status mage_append_block(const mage_kv_t *kv, const void *k_blk, const void *v_blk, int32_t *seq_lens, uint32_t *dev_status,
                              void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!k_blk || !v_blk || !seq_lens || kv->N_max < 1) return MAGE_ERR_INVALID_ARG;
    const KvView view = make_view(kv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int warps = kv->P * kv->H_kv * kv->B;
    append_rows_kernel<<<(warps + 3) / 4, 128, 0, st>>>(view, static_cast<const __nv_bfloat16 *>(k_blk), static_cast<const __nv_bfloat16 *>(v_blk),
                                                       seq_lens, dev_status);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    bump_seq_lens_kernel<<<(kv->P + 127) / 128, 128, 0, st>>>(view, seq_lens);
    return launch_check();
}

// Scratch for mage_exact_select_static.  In host code this name is only a handle for the runtime, not a device
// address: the address is looked up once per device below and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[MAGE_STATIC_SCRATCH_BYTES];
static void *g_static_scratch_addr[64] = {};      // per device, guarded by g_static_scratch_mu
static std::mutex g_static_scratch_mu;

mage_status mage_exact_select_static(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                                     float sm_scale, void *out, float *scores, uint32_t *dev_status, void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    const size_t need = make_plan(kv).exact_bytes;
    if (need > (size_t)MAGE_STATIC_SCRATCH_BYTES) {
        std::fprintf(stderr, "libmage: mage_exact_select_static needs %zu bytes of scratch for this description, the built-in "
                             "array holds %u; use mage_exact_select with a caller workspace\n", need, (unsigned)MAGE_STATIC_SCRATCH_BYTES);
        return MAGE_ERR_WORKSPACE;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MAGE_ERR_CUDA;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_scratch_mu);
        if (!g_static_scratch_addr[dev]) {  // set-up, once per device, with that device current
            void *addr = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&addr, g_static_scratch);
            if (e != cudaSuccess || !addr) {
                std::fprintf(stderr, "libmage: cudaGetSymbolAddress(static scratch) failed: %s\n", cudaGetErrorString(e));
                return MAGE_ERR_CUDA;
            }
            g_static_scratch_addr[dev] = addr;
        }
        scratch = g_static_scratch_addr[dev];
    }
    return mage_exact_select_events(kv, q, k_blk, v_blk, sm_scale, out, scores, scratch, (size_t)MAGE_STATIC_SCRATCH_BYTES,
                                    dev_status, stream, nullptr);
}

namespace {
struct PrunePlan {            // byte offsets into the workspace, after the exact pass's own part
    int tiles, seeds;         // key tiles per head (by N_max), seed tiles per head
    size_t rowsum, mass, seed_list, counts, compact, tau, list, list_count, total;
};
PrunePlan make_prune_plan(const mage_kv_t *kv, int k) {
    const Plan plan = make_plan(kv);
    const size_t heads = (size_t)kv->P * kv->H_kv;
    PrunePlan pp;
    pp.tiles = (kv->N_max + 127) / 128;
    // seed tiles: the heaviest eighth of a head's tiles, and at least twice the k keys the threshold needs.  They are scored in
    // any case; the threshold they give prunes the rest only if they hold at least k keys that stand out (otherwise it sits
    // at the background level, every tile passes it and the pass is the dense one)
    pp.seeds = std::min(pp.tiles, std::max(2 * ((k + 127) / 128), pp.tiles / 8));
    size_t off = plan.exact_bytes;
    auto take = [&](size_t bytes) { const size_t at = off; off += align_up(bytes, 256); return at; };
    pp.rowsum = take(heads * pp.tiles * plan.Mw * sizeof(float2));
    pp.mass = take(heads * pp.tiles * sizeof(float));
    pp.seed_list = take(heads * pp.seeds * sizeof(int));
    pp.counts = take((size_t)kv->P * 3 * sizeof(int));              // seed tiles taken, key tiles, entries of the compact rows: per problem
    pp.compact = take(heads * pp.seeds * 128 * sizeof(float));
    pp.tau = take(heads * sizeof(float));
    pp.list = take(heads * pp.tiles * sizeof(int));
    pp.list_count = take(heads * sizeof(int));
    pp.total = off;
    return pp;
}
}  // namespace

size_t mage_pruned_workspace_bytes(const mage_kv_t *kv, int32_t k) {
    if (!valid_kv(kv, nullptr) || k < 1) return 0;
    return make_prune_plan(kv, k).total;
}

mage_status mage_exact_select_pruned(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk, float sm_scale,
                                     int32_t k, float dense_above, void *out, float *scores, int32_t *indices, int32_t *k_eff,
                                     int32_t *tiles_scored, void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                                     void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (!q || !k_blk || !v_blk || !out || !indices || !k_eff || !workspace || k < 1 || (kv->N_max > 0 && !scores)) return MAGE_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f) || !(dense_above >= 0.f) || (reinterpret_cast<uintptr_t>(workspace) & 255)) return MAGE_ERR_INVALID_ARG;
    if (kv->flags & MAGE_FLAG_SIMT_KERNELS) return MAGE_ERR_UNSUPPORTED;
    const Plan plan = make_plan(kv);
    const PrunePlan pp = make_prune_plan(kv, k);
    if (workspace_bytes < pp.total) return MAGE_ERR_WORKSPACE;
    const KvView view = make_view(kv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int heads = kv->P * kv->H_kv;
    char *wsb = static_cast<char *>(workspace);
    float *ws = static_cast<float *>(workspace);
    const __nv_bfloat16 *qb = static_cast<const __nv_bfloat16 *>(q);
    if (kv->N_max == 0) {                                     // no prefix: attention inside the block, nothing to select
        const mage_status s = launch_exact_select(kv, view, plan, qb, static_cast<const __nv_bfloat16 *>(k_blk), static_cast<const __nv_bfloat16 *>(v_blk),
                                                  sm_scale, static_cast<__nv_bfloat16 *>(out), nullptr, ws, dev_status, st, nullptr);
        if (s != MAGE_OK) return s;
        if (tiles_scored && cudaMemsetAsync(tiles_scored, 0, (size_t)heads * sizeof(int), st) != cudaSuccess) return MAGE_ERR_CUDA;
        topk_kernel<<<heads, kTopkThreads, 0, st>>>(scores, kv->seq_lens, kv->H_kv, 0, k, indices, k_eff);
        return launch_check();
    }
    // the score pass's tensor maps first: nothing is launched if they cannot be encoded
    CUtensorMap map_q_rows, map_k;
    const mage_status sup = tc_supported(kv);
    if (sup != MAGE_OK) return sup;
    if (!tc::make_rows_map(&map_q_rows, q, (long long)kv->P * kv->H_q * kv->B) || !tc::make_cache_map(&map_k, kv, kv->k_cache)) return MAGE_ERR_UNSUPPORTED;
    float2 *rowsum = reinterpret_cast<float2 *>(wsb + pp.rowsum);
    float *mass = reinterpret_cast<float *>(wsb + pp.mass), *compact = reinterpret_cast<float *>(wsb + pp.compact), *tau = reinterpret_cast<float *>(wsb + pp.tau);
    int *seed_list = reinterpret_cast<int *>(wsb + pp.seed_list), *seed_count = reinterpret_cast<int *>(wsb + pp.counts), *tile_counts = seed_count + kv->P,
        *compact_lens = seed_count + 2 * kv->P, *list = reinterpret_cast<int *>(wsb + pp.list), *list_count = reinterpret_cast<int *>(wsb + pp.list_count);
    // 1. exact attention; the pass also leaves each tile's row sums behind
    mage_status s = launch_exact_select(kv, view, plan, qb, static_cast<const __nv_bfloat16 *>(k_blk), static_cast<const __nv_bfloat16 *>(v_blk), sm_scale,
                                        static_cast<__nv_bfloat16 *>(out), nullptr, ws, dev_status, st, nullptr, false, rowsum, pp.tiles);
    if (s != MAGE_OK) return s;
    // 2. tile masses, 3. the seed tiles = the largest masses
    const long long warps = (long long)heads * pp.tiles;
    prune::tile_mass_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(view, plan, rowsum, pp.tiles, ws, mass, tile_counts);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    topk_kernel<<<heads, kTopkThreads, 0, st>>>(mass, tile_counts, kv->H_kv, pp.tiles, pp.seeds, seed_list, seed_count);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    // 4. exact scores of the seed tiles (also in list order, for the threshold)
    const float scale_log2 = sm_scale * kLog2e;
    const int tpc_dense = tc::tiles_per_cta_for(heads, kv->N_max, kv->page_size != 0), tpc = std::max(1, std::min(32, tpc_dense));
    tc::ScoreTileList seeds;
    seeds.tiles = seed_list; seeds.count = seed_count; seeds.stride = pp.seeds; seeds.count_per_problem = 1;
    seeds.compact = compact; seeds.compact_lens = compact_lens;
    if (launch_score_pass(view, plan, map_q_rows, map_k, (pp.seeds + tpc - 1) / tpc, tpc, scale_log2, ws, scores, dev_status, st, seeds) != MAGE_OK) return MAGE_ERR_CUDA;
    // 5. tau = the k-th largest seed score (0 if the seeds hold no more than k keys: then nothing is pruned)
    topk_kernel<<<heads, kTopkThreads, 0, st>>>(compact, compact_lens, kv->H_kv, pp.seeds * 128, k, indices, k_eff, tau);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    // 6. the further tiles to score; zeros where nothing can be selected
    prune::mark_kernel<<<heads, 256, (size_t)pp.tiles, st>>>(view, pp.tiles, mass, seed_list, pp.seeds, seed_count, tau, dense_above, list, list_count, scores, tiles_scored);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    // 7. their exact scores, 8. Top-k of the array
    tc::ScoreTileList rest;
    rest.tiles = list; rest.count = list_count; rest.stride = pp.tiles;
    if (launch_score_pass(view, plan, map_q_rows, map_k, (pp.tiles + tpc - 1) / tpc, tpc, scale_log2, ws, scores, dev_status, st, rest) != MAGE_OK) return MAGE_ERR_CUDA;
    topk_kernel<<<heads, kTopkThreads, 0, st>>>(scores, kv->seq_lens, kv->H_kv, kv->N_max, k, indices, k_eff);
    return launch_check();
}

size_t mage_quest_workspace_bytes(const mage_kv_t *kv, int32_t k) {
    if (!valid_kv(kv, nullptr) || k < MAGE_QUEST_PAGE || k % MAGE_QUEST_PAGE) return 0;
    // page counts [P], selected-page counts [P], selected pages [P][H_kv][k/16]
    return align_up((size_t)kv->P * 2 * sizeof(int), 256) + align_up((size_t)kv->P * kv->H_kv * (k / MAGE_QUEST_PAGE) * sizeof(int), 256);
}

mage_status mage_quest_build(const mage_kv_t *kv, void *page_min, void *page_max, uint32_t *dev_status, void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (kv->page_size % MAGE_QUEST_PAGE) return MAGE_ERR_UNSUPPORTED;
    if (kv->N_max < MAGE_QUEST_PAGE) return MAGE_OK;              // no whole page anywhere
    if (!page_min || !page_max) return MAGE_ERR_INVALID_ARG;
    const KvView view = make_view(kv);
    const int n_pages_max = (kv->N_max + MAGE_QUEST_PAGE - 1) / MAGE_QUEST_PAGE;
    const long long warps = (long long)kv->P * kv->H_kv * n_pages_max;
    quest::build_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(view, n_pages_max, static_cast<__nv_bfloat16 *>(page_min),
                                                                                                  static_cast<__nv_bfloat16 *>(page_max), dev_status);
    return launch_check();
}

mage_status mage_quest_select(const mage_kv_t *kv, const void *q, const void *page_min, const void *page_max, int32_t k,
                              float *page_scores, int32_t *indices, int32_t *k_eff, void *workspace, size_t workspace_bytes,
                              void *stream) {
    mage_status why = MAGE_OK;
    if (!valid_kv(kv, &why)) return why;
    if (k < MAGE_QUEST_PAGE || k % MAGE_QUEST_PAGE || !q || !indices || !k_eff || !workspace || (reinterpret_cast<uintptr_t>(workspace) & 255)) return MAGE_ERR_INVALID_ARG;
    if (kv->page_size % MAGE_QUEST_PAGE) return MAGE_ERR_UNSUPPORTED;
    if (workspace_bytes < mage_quest_workspace_bytes(kv, k)) return MAGE_ERR_WORKSPACE;
    const int n_pages_max = (kv->N_max + MAGE_QUEST_PAGE - 1) / MAGE_QUEST_PAGE;
    if (n_pages_max > 0 && (!page_min || !page_max || !page_scores)) return MAGE_ERR_INVALID_ARG;
    const KvView view = make_view(kv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int heads = kv->P * kv->H_kv, k_pages = k / MAGE_QUEST_PAGE;
    int *page_counts = static_cast<int *>(workspace), *pages_sel = page_counts + kv->P;
    int *page_idx = reinterpret_cast<int *>(static_cast<char *>(workspace) + align_up((size_t)kv->P * 2 * sizeof(int), 256));
    quest::score_kernel<<<dim3(std::max(1, (n_pages_max + quest::kPagesPerCta - 1) / quest::kPagesPerCta), heads), 256, 0, st>>>(
        view, n_pages_max, static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(page_min),
        static_cast<const __nv_bfloat16 *>(page_max), page_scores, page_counts);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    topk_kernel<<<heads, kTopkThreads, 0, st>>>(page_scores, page_counts, kv->H_kv, n_pages_max, k_pages, page_idx, pages_sel);
    if (launch_check() != MAGE_OK) return MAGE_ERR_CUDA;
    quest::expand_kernel<<<heads, 256, 0, st>>>(kv->H_kv, k, page_idx, pages_sel, indices, k_eff);
    return launch_check();
}

const char *mage_status_string(mage_status s) {
    switch (s) {
        case MAGE_OK: return "MAGE_OK";
        case MAGE_ERR_INVALID_ARG: return "MAGE_ERR_INVALID_ARG";
        case MAGE_ERR_UNSUPPORTED: return "MAGE_ERR_UNSUPPORTED";
        case MAGE_ERR_WORKSPACE: return "MAGE_ERR_WORKSPACE";
        case MAGE_ERR_CUDA: return "MAGE_ERR_CUDA";
    }
    return "MAGE_ERR_UNKNOWN";
}

uint64_t mage_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

#ifdef MAGE_TIMING
int mage_debug_topk_stamps(unsigned long long *host_out) { return (int)cudaMemcpyFromSymbol(host_out, g_topk_stamps, sizeof(unsigned long long) * 64); }
int mage_debug_stamps(unsigned long long *host_out) { return (int)cudaMemcpyFromSymbol(host_out, tc::g_stamps, sizeof(unsigned long long) * 128); }
#endif

}  // extern "C"

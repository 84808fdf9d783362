/*
 * libmage -- the per-block sparse-attention hot path of MAGE ([MASK]-Guided
 * Sparse Attention for block-diffusion LLMs) for NVIDIA B200 (sm_100a).
 *
 * Three stages, one entry point each (paper: Algorithm 1 and Section 4):
 *
 *   mage_exact_select       Step 1 of a block (Phase 1): exact attention of the
 *                           all-[MASK] block over the whole prefix KV cache plus
 *                           the block's own keys, and, in the same call, the
 *                           per-block score of every prefix position (Eq. 4).
 *   mage_topk               per-KV-head Top-k of those scores (Eq. 4 / Eq. 2),
 *                           meant to be enqueued on a side ("select") stream.
 *   mage_sparse_block_attn  steps 2..T (Phase 2): attention over the k selected
 *                           cache rows plus the block's own keys, one softmax.
 *
 * Notation (paper, Section 3.1): H_q query heads, H_kv KV heads, G = H_q/H_kv
 * query heads per KV head with group(h) = {hG .. hG+G-1}, B tokens per block,
 * N prefix length, d head dimension, k budget.  A batch holds P independent
 * problems (layers of one model, or sequences of a serving batch).
 *
 * Conventions
 *   - Plain C ABI.  Every pointer argument except the mage_kv_t itself is DEVICE
 *     memory owned by the caller; the library allocates nothing and keeps no
 *     state between calls.  `stream` is a cudaStream_t passed as void*.
 *   - All calls only enqueue work on `stream` and return.  The return value
 *     covers host-detectable errors; nothing is launched when it is not MAGE_OK.
 *     The tensor-core kernels are launched with the programmatic stream
 *     serialization attribute and wait for their predecessor before they touch
 *     global memory: ordering against other work in the stream is that of
 *     ordinary stream order, and the calls may be captured into a CUDA graph.
 *   - Device-detectable problems (an index outside [0, N_p), a page id outside
 *     [0, num_pages), a bounded wait that expired) set bits in *dev_status
 *     (optional, may be NULL) and the offending access is skipped; a kernel
 *     never traps.
 *   - bf16 tensors are row-major with the head dimension contiguous; the score
 *     and all accumulation are fp32.
 */
#ifndef MAGE_H_
#define MAGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MAGE_OK = 0,
    MAGE_ERR_INVALID_ARG = -1,  /* null pointer, bad shape, k < 1, ...              */
    MAGE_ERR_UNSUPPORTED = -2,  /* valid but not built: d != 128, B > 64, ...       */
    MAGE_ERR_WORKSPACE = -3,    /* workspace smaller than mage_workspace_bytes()   */
    MAGE_ERR_CUDA = -4          /* a CUDA call failed while enqueueing              */
} mage_status;

/* bits of *dev_status */
#define MAGE_DEV_BAD_INDEX 1u   /* indices[] entry outside [0, N_p): row skipped    */
#define MAGE_DEV_BAD_PAGE 2u    /* block_table entry outside [0, num_pages): skipped */
#define MAGE_DEV_TIMEOUT 4u     /* an in-kernel bounded wait gave up                */
#define MAGE_DEV_CACHE_FULL 8u  /* mage_append_block: no room left for the block: nothing appended for that problem */

/* mage_kv_t.flags */
#define MAGE_FLAG_SIMT_KERNELS 1  /* use the portable CUDA-core kernels for every stage (about 25x slower; for cross-checks
                                     and for layouts the tensor-core kernels do not take).  The library never switches to
                                     them by itself: without this flag, a description that the tensor-core kernels cannot
                                     take is refused with MAGE_ERR_UNSUPPORTED and nothing is launched.  That concerns:
                                     page sizes that are not multiples of 64, k_cache / v_cache (or, in the reuse step,
                                     k_blk / v_blk) not 16-byte aligned, strides or extents that a TMA tensor map cannot
                                     express, and, in the reuse step on a cache that is not one list of rows with a single
                                     pitch, a cache of more than 2^34 elements. */

#define MAGE_FLAG_TEST_STALL 2    /* test hook for the bounded waits: the exact pass of mage_exact_select / mage_exact_attn /
                                     mage_select_scores never requests its first key tile, and every wait in that kernel
                                     gives up after about 1 ms instead of 0.25 s.  The call still returns normally:
                                     MAGE_DEV_TIMEOUT is set in *dev_status, outputs and scores are undefined, nothing is
                                     left in flight, and the context stays usable.  Not for production use. */

/*
 * Prefix KV cache "C" of Algorithm 1 for a batch of P problems, read-only.
 *
 * Contiguous (page_size == 0): element (p, h, j, c) of K is
 *     k_cache[p*stride_p + h*stride_h + j*stride_n + c]     (strides in elements, c < d contiguous)
 * and likewise for V.  Strides must be multiples of 8 elements.
 * Paged (page_size > 0): k_cache / v_cache are pools [num_pages][H_kv][page_size][d];
 * logical position j of problem p lives in pool page block_table[p*max_pages + j/page_size],
 * row j % page_size.  Strides are ignored.
 * seq_lens[p] = N_p <= N_max is the prefix length of problem p (NULL: every N_p = N_max).
 * N_p = 0 is legal.  Cache rows at positions >= N_p are never used as data.  P * H_kv <= 65535.
 */
typedef struct mage_kv {
    int32_t P, H_q, H_kv, d;      /* d must be 128; H_q % H_kv == 0                    */
    int32_t B;                    /* 1..64 block tokens                                */
    int32_t page_size;            /* 0 = contiguous, else tokens per page (power of two >= 16; see MAGE_FLAG_SIMT_KERNELS) */
    const void *k_cache, *v_cache;
    int64_t stride_p, stride_h, stride_n;
    const int32_t *block_table;   /* device [P][max_pages], paged only                 */
    int32_t max_pages, num_pages;
    const int32_t *seq_lens;      /* device [P] or NULL                                */
    int32_t N_max;                /* host-known bound on N_p; row stride of `scores`   */
    int32_t flags;                /* MAGE_FLAG_*                                       */
} mage_kv_t;

/*
 * Bytes of device workspace that any call on this cache description needs
 * (host-only arithmetic, no CUDA call).  k_max is the largest budget that will
 * be passed.  Returns 0 for an invalid description.  The workspace must be
 * 256-byte aligned; its contents need not be preserved between calls, and two
 * calls that may overlap on the GPU need separate workspaces.
 */
size_t mage_workspace_bytes(const mage_kv_t *kv, int32_t k_max);

/*
 * Step 1 of a block: exact attention + block score (Algorithm 1, Phase 1:
 * main-stream "Attn(Q, K, V, C)" and select-stream "A = softmax(Q K^T / sqrt d)",
 * "alpha = 1/(GB) sum_{g,q} A[g,q,:]"; Eq. 4).
 *
 *   q      [P][H_q][B][d]  bf16   queries of the all-[MASK] block
 *   k_blk  [P][H_kv][B][d] bf16   the block's own keys  (attended densely, no mask, self included)
 *   v_blk  [P][H_kv][B][d] bf16   the block's own values
 *   out    [P][H_q][B][d]  bf16   softmax over the N_p prefix keys and the B block keys, times V
 *   scores [P][H_kv][N_max] fp32  scores[p][h][j] = 1/(G*B) * sum over g in group(h), q of
 *                                 softmax_j over the PREFIX keys of sm_scale * <q[g][q], K[h][j]>,
 *                                 for j < N_p; entries j >= N_p are left untouched.
 *   sm_scale  applied in fp32 to the accumulated dot product (1/sqrt(d) in the paper)
 */
mage_status mage_exact_select(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                              float sm_scale, void *out, float *scores, void *workspace, size_t workspace_bytes,
                              uint32_t *dev_status, void *stream);

/*
 * The same operation as mage_exact_select (Algorithm 1, Phase 1; Eq. 4), with
 * CUDA events recorded between its kernels so that a caller can time each one
 * on the stream it runs on.  `events` is a HOST array of 4 cudaEvent_t handles
 * (created by the caller with timing enabled), recorded on `stream` in this order:
 *   [0] before the first kernel, [1] after the attention kernel over prefix + block keys,
 *   [2] after the kernel that merges the per-chunk partial results,
 *   [3] after the block-score kernel.
 * events == NULL behaves exactly like mage_exact_select.
 */
mage_status mage_exact_select_events(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                                     float sm_scale, void *out, float *scores, void *workspace,
                                     size_t workspace_bytes, uint32_t *dev_status, void *stream, void **events);

/*
 * Top-k selection per KV head (Algorithm 1, "S <- Top-k(alpha)"; Eq. 4).
 *
 *   scores   [P][H_kv][N_max] fp32, non-negative, no NaN
 *   indices  [P][H_kv][k] int32   the k_eff = min(k, N_p) positions with the largest score, in
 *                                 ascending position order; equal scores go to the smaller position;
 *                                 slots >= k_eff are set to -1
 *   k_eff    [P] int32            min(k, N_p)
 * Exact (a radix select on the fp32 bit patterns), deterministic.  Needs no
 * workspace (the arguments are kept for symmetry; they may be NULL / 0).
 */
mage_status mage_topk(const float *scores, const int32_t *seq_lens, int32_t P, int32_t H_kv, int32_t N_max,
                      int32_t k, int32_t *indices, int32_t *k_eff, void *workspace, size_t workspace_bytes,
                      void *stream);

/*
 * Reuse step, run at each of the T-1 remaining denoising steps (Algorithm 1,
 * Phase 2, "SparseAttn(Q, K, V, C[S])").
 *
 *   q, k_blk, v_blk, out   as in mage_exact_select, holding the current step's tensors
 *   indices [P][H_kv][k] int32, k_eff [P] int32   as written by mage_topk.  Any order is accepted;
 *       a position listed twice is attended twice.  The same tensors serve every step of the block
 *       (the selection is fixed at Step 1), so they must stay alive and unmodified until the last
 *       reuse step has run.
 * Each query attends to cache rows indices[p][h][0 .. k_eff[p]-1] of its KV head and to all B
 * block keys, in one softmax.  With k_eff = N_p the result equals the exact pass.
 */
mage_status mage_sparse_block_attn(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                                   const int32_t *indices, const int32_t *k_eff, int32_t k, float sm_scale,
                                   void *out, void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                                   void *stream);

/*
 * End of a block (Algorithm 1, last line: "C <- C || KV(x)"): append the finished block's keys and values to the
 * prefix cache, so that the next block sees a prefix of N_p + B tokens.
 *
 *   k_blk, v_blk [P][H_kv][B][d] bf16   the block's final keys / values
 *   seq_lens     [P] int32, device, in/out   N_p on entry, N_p + B on return (this argument, not kv->seq_lens, is
 *                                            what is read and updated; it may be the same array)
 * Rows go to logical positions N_p .. N_p+B-1: contiguous layout needs N_p + B <= N_max; paged layout needs the
 * block table to map the pages those positions fall in already (the caller owns page allocation).  A problem that
 * has no room, or whose page id is out of range, is left unchanged and MAGE_DEV_CACHE_FULL / MAGE_DEV_BAD_PAGE is
 * set in *dev_status.  This is the one call that writes through kv->k_cache / kv->v_cache.
 */
mage_status mage_append_block(const mage_kv_t *kv, const void *k_blk, const void *v_blk, int32_t *seq_lens,
                              uint32_t *dev_status, void *stream);

/*
 * The main stream's half of Step 1 on its own (Algorithm 1, main stream:
 * "Attn(Q, K, V, C)"): exact attention of the block over the prefix cache and its
 * own keys, no block scores.  Arguments, layouts and errors as mage_exact_select
 * (which is this call followed by the score pass, sharing the rows' log-sum-exp).
 */
mage_status mage_exact_attn(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk, float sm_scale,
                            void *out, void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream);

/*
 * The select stream's computation on its own (Algorithm 1, select stream:
 * "A = softmax(Q K^T / sqrt d)" over the prefix cache, then Eq. 4's mean over the
 * block's G*B rows), without the attention output: block scores from the queries
 * and the cached keys alone.  For callers that run the selection beside the main
 * stream's attention as the paper does, rather than reuse mage_exact_select's pass.
 * Work: one pass over K for the rows' log-sum-exp (no V, no block keys), one pass
 * for the scores.  The scores are bit-identical to mage_exact_select's.
 *
 *   q          [P][H_q][B][d] bf16, device.
 *   scores     [P][H_kv][N_max] fp32, device, written for positions < N_p; may be
 *              NULL only when N_max == 0.
 *   workspace  device, 256-byte aligned, at least mage_workspace_bytes(kv, k_max)
 *              for any k_max >= 1; it must not be the workspace of a call that may
 *              run at the same time on another stream.
 * Errors: as mage_exact_select.
 */
mage_status mage_select_scores(const mage_kv_t *kv, const void *q, float sm_scale, float *scores, void *workspace,
                               size_t workspace_bytes, uint32_t *dev_status, void *stream);

/*
 * Step 1 of a block for callers that cannot hand over a workspace (the paper has no counterpart; this is a
 * packaging variant of mage_exact_select, same arithmetic, same kernels).
 *
 * Some hosts of this library may not allocate device memory at the point where they call it: an inference
 * runtime that carves up all of its memory at start-up and forbids cudaMalloc afterwards, a plugin that runs
 * inside someone else's memory pool, code on a latency path where an allocation would stall the device.  For
 * them this entry point takes no workspace argument: the partial results and per-row normalisers that
 * mage_exact_select keeps in the caller's workspace live in an array that is part of the library image itself
 * (a file-scope __device__ array of MAGE_STATIC_SCRATCH_BYTES = 32 MiB, held by every GPU that loads the library
 * until the process exits).  Inputs and outputs are still the caller's.
 *
 *   - A description whose mage_workspace_bytes() exceeds MAGE_STATIC_SCRATCH_BYTES is rejected with
 *     MAGE_ERR_WORKSPACE (and a line on stderr); nothing is launched.  As a guide, one Qwen2.5-7B-shaped layer
 *     with a 32K-token prefix needs about 18 MB; a 28-layer 128K batch does not fit.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *     current) and remembers it; make that first call outside any stream capture.  The remembered address does
 *     not survive a cudaDeviceReset of that device: do not reset a device between calls of this entry point.
 *   - The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - All calls on a device share the one array, which simply keeps whatever the last call left in it.  Nothing
 *     in it has to start at zero: the kernels write every element they later read.  Two calls that can overlap
 *     on the GPU (different streams, no ordering between them) would race on it; order them.
 */
#define MAGE_STATIC_SCRATCH_BYTES (32u << 20)
mage_status mage_exact_select_static(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk,
                                     float sm_scale, void *out, float *scores, uint32_t *dev_status, void *stream);

/*
 * Step 1 and the selection in one call, scoring only where a selected key can be (Algorithm 1, Phase 1: main-stream
 * "Attn(Q, K, V, C)", select-stream "alpha", "S <- Top-k(alpha)"; Eq. 4).  The result -- out, indices, k_eff -- is that
 * of mage_exact_select followed by mage_topk; what differs is the work: the exact pass records, per 128-key tile and
 * query row, the probability mass the row puts on the tile; a key's score is at most its tile's mass averaged over
 * rows; tiles whose mass is below the k-th largest exact score found among the heaviest tiles cannot hold a selected key
 * and are not scored (their entries of `scores` are written as 0).  On flat attention every tile is scored, as in
 * mage_exact_select; on concentrated attention the second pass over K shrinks to the tiles that matter.
 *
 *   k            budget, as in mage_topk
 *   dense_above  when more than this fraction (0..1) of a head's remaining tiles would be scored anyway, all of them are
 *   scores       [P][H_kv][N_max] fp32: exact (Eq. 4) in scored tiles, 0 elsewhere below N_p; untouched from N_p on
 *   indices, k_eff  as mage_topk writes them
 *   tiles_scored [P][H_kv] int32, optional (may be NULL): key tiles of each head that went through the score pass
 *   workspace    device, 256-byte aligned, at least mage_pruned_workspace_bytes(kv, k)
 * Runs on `stream` only.  Not available with MAGE_FLAG_SIMT_KERNELS (MAGE_ERR_UNSUPPORTED).
 */
size_t mage_pruned_workspace_bytes(const mage_kv_t *kv, int32_t k);
mage_status mage_exact_select_pruned(const mage_kv_t *kv, const void *q, const void *k_blk, const void *v_blk, float sm_scale,
                                     int32_t k, float dense_above, void *out, float *scores, int32_t *indices, int32_t *k_eff,
                                     int32_t *tiles_scored, void *workspace, size_t workspace_bytes, uint32_t *dev_status,
                                     void *stream);

/*
 * Quest-style page estimator in its per-block form: the paper's comparison system on the same inputs, not a part of
 * MAGE (Section 2.2: pages of p tokens summarised by per-channel max / min keys, page score = the sign-aware upper
 * bound sum_c max(q_c Kmax_c, q_c Kmin_c) on q.k; Section 3.1, Eq. 2 with that estimate as s: the mean over the
 * block's G*B queries; Section 5, Setup: p = 16, re-estimated at every denoising step).
 *
 * mage_quest_build summarises the whole pages of every prefix (positions [0, 16*floor(N_p/16)); a ragged tail of
 * fewer than 16 tokens is never a candidate):
 *   page_min, page_max  [P][H_kv][ceil(N_max/16)][d] bf16, device, written for whole pages only
 * mage_quest_select scores the pages against the current queries, takes the k/16 best pages per KV head (exact,
 * ties to the smaller page) and writes their tokens as an index set that mage_sparse_block_attn accepts:
 *   q            [P][H_q][B][d] bf16
 *   k            a multiple of 16
 *   page_scores  [P][H_kv][ceil(N_max/16)] fp32, written for whole pages
 *   indices      [P][H_kv][k] int32 ascending, -1 padded;  k_eff [P] int32 = 16 * min(k/16, floor(N_p/16))
 *   workspace    device, 256-byte aligned, at least mage_quest_workspace_bytes(kv, k)
 * Cache page sizes must be multiples of 16 (or 0).  Errors as the other calls; nothing is launched unless MAGE_OK.
 */
#define MAGE_QUEST_PAGE 16
size_t mage_quest_workspace_bytes(const mage_kv_t *kv, int32_t k);
mage_status mage_quest_build(const mage_kv_t *kv, void *page_min, void *page_max, uint32_t *dev_status, void *stream);
mage_status mage_quest_select(const mage_kv_t *kv, const void *q, const void *page_min, const void *page_max, int32_t k,
                              float *page_scores, int32_t *indices, int32_t *k_eff, void *workspace, size_t workspace_bytes,
                              void *stream);

/*
 * Keys and queries in 8 bits (e4m3) for Step 1 and the reuse step.  The paper leaves the compression of the cache to
 * future work (Limitations); this variant is the library's own, defined as the unchanged method (Algorithm 1; Eq. 4)
 * applied to de-quantised queries and keys:
 *
 *   scale    one per (problem, KV head): s = amax / 448 in single precision (1 when amax = 0), amax the largest |x| of the
 *            head's rows -- the cached keys below N_p for s_k; the G*B query rows of the call for s_q, taken at every call
 *   code     e4m3 (1 sign, 4 exponent, 3 mantissa bits; largest value 448, no infinities) of x / s: IEEE single division,
 *            round to nearest even, magnitudes beyond 448 clamp to 448
 *   keys     cached keys and the block's own keys use the head's s_k (block keys larger than the cache's amax clamp)
 *   logits   s_q s_k * (code_q . code_k), accumulated in fp32 by the tensor cores; values, probabilities and outputs are
 *            as in the 16-bit calls.  The key bytes read from the cache halve (128 instead of 256 per token and head, in
 *            both passes of Step 1 and in the gather of the reuse step); the value bytes do not change.
 *
 * mage_k8_quantize_cache writes the codes of cache rows [row_begin, N_p) of every (problem, KV head):
 *   k8_cache   device, 16-byte aligned: one byte per element, addressed exactly like kv->k_cache (same strides in
 *              elements, same page table), so it is as large in elements as the key cache
 *   k_scale    [P][H_kv] fp32, device.  row_begin = 0: written (from the rows below N_p); row_begin > 0: read -- rows
 *              appended later are coded under the scale the head already has
 *   Contiguous caches need strides that are multiples of 16 elements.
 * mage_exact_select_k8 / mage_sparse_block_attn_k8 are mage_exact_select / mage_sparse_block_attn with the keys taken from
 * the codes: kv->k_cache is not read (it may be NULL); kv->v_cache, q, k_blk, v_blk, the outputs and the workspace are as
 * there.  The queries and block keys of a call are coded on the way: by one small kernel in front, into k8->scratch, for
 * Step 1 and for a reuse step with more than 256 query rows per KV head; inside the kernel for the other reuse steps.
 *   k8->scratch  device, 256-byte aligned, at least mage_k8_scratch_bytes(kv); contents are per call
 * Not available with MAGE_FLAG_SIMT_KERNELS, and the reuse step needs a cache that is one list of rows with a single pitch
 * (every paged pool; contiguous layouts whose head and problem strides are multiples of the row stride): otherwise
 * MAGE_ERR_UNSUPPORTED.  Errors as the other calls; nothing is launched unless MAGE_OK.
 */
typedef struct mage_k8 {
    const void *k8_cache;  /* device: e4m3 codes of the keys                                  */
    const float *k_scale;  /* device [P][H_kv]: de-quantisation scale of each head's keys      */
    void *scratch;         /* device: codes of the call's queries and block keys, s_q s_k     */
} mage_k8_t;
size_t mage_k8_scratch_bytes(const mage_kv_t *kv);
mage_status mage_k8_quantize_cache(const mage_kv_t *kv, int32_t row_begin, void *k8_cache, float *k_scale, uint32_t *dev_status,
                                   void *stream);
mage_status mage_exact_select_k8(const mage_kv_t *kv, const mage_k8_t *k8, const void *q, const void *k_blk, const void *v_blk,
                                 float sm_scale, void *out, float *scores, void *workspace, size_t workspace_bytes,
                                 uint32_t *dev_status, void *stream);
/* The same call with four caller events recorded between its kernels, as mage_exact_select_events (the block-code kernel
 * falls between events[0] and events[1], with the exact pass). */
mage_status mage_exact_select_k8_events(const mage_kv_t *kv, const mage_k8_t *k8, const void *q, const void *k_blk, const void *v_blk,
                                        float sm_scale, void *out, float *scores, void *workspace, size_t workspace_bytes,
                                        uint32_t *dev_status, void *stream, void **events);
mage_status mage_sparse_block_attn_k8(const mage_kv_t *kv, const mage_k8_t *k8, const void *q, const void *k_blk, const void *v_blk,
                                      const int32_t *indices, const int32_t *k_eff, int32_t k, float sm_scale, void *out,
                                      void *workspace, size_t workspace_bytes, uint32_t *dev_status, void *stream);

/* Static, human-readable name of a status code. */
const char *mage_status_string(mage_status s);

/* Number of kernels the library has launched in this process (for bookkeeping in benchmarks). */
uint64_t mage_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MAGE_H_ */

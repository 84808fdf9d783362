// Pruned exact selection: the block scores (Eq. 4) are only computed where a selected key can be.
//
// Every term of score[j] = 1/(G B) * sum_r softmax_r[j] is positive, so the score of a key is at most the probability
// mass that the rows put on the whole 128-key tile the key lies in, averaged over rows:
//     score[j] <= mass[tile(j)] = 1/(G B) * sum_r sum_{j' in tile} softmax_r[j'].
// The exact pass already forms sum_{j' in tile} exp2(s_rj' - reference_r) for its own row sums; it writes those per
// (tile, row) with the reference, and once the rows' log-sum-exp is known the masses follow without touching K again.
// With tau = the k-th largest exact score among any set of at least k scored keys, a tile whose mass is below tau holds
// no selected key.  So: score the tiles with the largest masses, take tau from them, score every other tile whose mass
// reaches tau, and leave the rest at zero -- the Top-k of that array is the Top-k of the full exact score array.
// On flat attention (every tile's mass far above tau) nothing is pruned and every tile is scored, as in the dense pass.
#pragma once
#include "common.cuh"

namespace mage {
namespace prune {

constexpr int kTileKeys = 128;
constexpr float kMassMargin = 0.99f;     // masses and tau are fp32 results (and, after an in-tile reference jump, carry a
                                         // bf16-rounded half): a tile is kept unless its mass is below 0.99 * tau

// One warp per (problem, KV head, tile): mass = 1/M * sum_r rowsum[r] * 2^(reference[r] - lse2[r]).
__global__ void __launch_bounds__(256) tile_mass_kernel(KvView kv, Plan plan, const float2 *__restrict__ rowsum, int tiles_max,
                                                        const float *__restrict__ ws, float *__restrict__ mass, int *__restrict__ tile_counts) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (long long)kv.P * kv.H_kv * tiles_max) return;
    const int tile = (int)(warp % tiles_max), z = (int)(warp / tiles_max), p = z / kv.H_kv;
    const int tiles = (seq_len_of(kv, p) + kTileKeys - 1) / kTileKeys;
    if (tile == 0 && z % kv.H_kv == 0 && lane == 0) tile_counts[p] = tiles;
    if (tile >= tiles) return;
    const float2 *rs = rowsum + ((size_t)z * tiles_max + tile) * plan.Mw;
    const float *neg_lse = ws + plan.off_neg_lse + (size_t)z * plan.Mw;
    float acc = 0.f;
    for (int r = lane; r < kv.M; r += 32) {
        const float2 v = rs[r];
        acc += v.x * exp2f(v.y + neg_lse[r]);
    }
#pragma unroll
    for (int w = 16; w; w >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, w);
    if (lane == 0) mass[(size_t)z * tiles_max + tile] = acc / (float)kv.M;
}

// CTA = (problem, KV head).  From the masses, the seed tiles already scored and tau (the k-th largest seed score, 0 when
// the seeds hold fewer than k keys): the ascending list of further tiles to score -- those whose mass reaches tau, or every
// remaining tile when more than `dense_above` of them would be listed anyway -- and zeros in the score array for the
// tiles that are neither seeds nor listed.  tiles_scored (optional) receives seeds + listed per head.
__global__ void __launch_bounds__(256) mark_kernel(KvView kv, int tiles_max, const float *__restrict__ mass, const int *__restrict__ seeds,
                                                   int seed_stride, const int *__restrict__ seed_count, const float *__restrict__ tau,
                                                   float dense_above, int *__restrict__ list, int *__restrict__ list_count,
                                                   float *__restrict__ scores, int *__restrict__ tiles_scored) {
    extern __shared__ unsigned char flag[];               // per tile: 2 = seed, 1 = listed, 0 = pruned
    __shared__ int warp_tot[8], n_cand_s, run_s;
    const int z = blockIdx.x, p = z / kv.H_kv, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = seq_len_of(kv, p), tiles = (N + kTileKeys - 1) / kTileKeys;
    const int n_seed = min(seed_count[p], seed_stride);
    const float thr = tau[z] * kMassMargin;
    if (tid == 0) { n_cand_s = 0; run_s = 0; }
    for (int t = tid; t < tiles; t += 256) flag[t] = mass[(size_t)z * tiles_max + t] >= thr ? 1 : 0;
    __syncthreads();
    for (int i = tid; i < n_seed; i += 256) flag[seeds[(size_t)z * seed_stride + i]] = 2;
    __syncthreads();
    int mine = 0;
    for (int t = tid; t < tiles; t += 256) mine += flag[t] == 1;
    mine = __reduce_add_sync(0xffffffffu, mine);
    if (lane == 0) atomicAdd(&n_cand_s, mine);
    __syncthreads();
    const bool dense = (float)n_cand_s > dense_above * (float)(tiles - n_seed);
    if (dense)
        for (int t = tid; t < tiles; t += 256)
            if (flag[t] == 0) flag[t] = 1;
    __syncthreads();
    // ordered compaction of the listed tiles, 256 tiles at a time
    for (int base = 0; base < tiles; base += 256) {
        const int t = base + tid;
        const int f = t < tiles && flag[t] == 1;
        const unsigned bal = __ballot_sync(0xffffffffu, f);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = run_s;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (f) list[(size_t)z * tiles_max + before + __popc(bal & ((1u << lane) - 1u))] = t;
        __syncthreads();
        if (tid == 0) { int tot = 0; for (int w = 0; w < 8; ++w) tot += warp_tot[w]; run_s += tot; }
        __syncthreads();
    }
    if (tid == 0) {
        list_count[z] = run_s;
        if (tiles_scored) tiles_scored[z] = run_s + n_seed;
    }
    // pruned tiles: their scores are below tau, whatever they are; the array holds zeros there
    float *srow = scores + (size_t)z * kv.N_max;
    for (int t = 0; t < tiles; ++t) {
        if (flag[t] != 0) continue;
        const int j = t * kTileKeys + tid;
        if (tid < kTileKeys && j < N) srow[j] = 0.f;
    }
}

}  // namespace prune
}  // namespace mage

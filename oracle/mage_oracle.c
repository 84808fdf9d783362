/*
 * CPU oracle for the MAGE per-block attention path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, by-definition implementations in fp64 of what the CUDA library
 * computes.  Nothing here is tiled, fused, split or reordered, and nothing is
 * shared with the CUDA code: the tests, the smoke check and the benchmark's CPU
 * baseline are the only callers.  Inputs are fp32 arrays holding bf16-exact
 * values (the same bit patterns the GPU gets); all arithmetic is double.
 *
 * Notation follows the paper: H_q query heads, H_kv KV heads, G = H_q / H_kv
 * query heads per KV head, group(h) = {hG .. hG+G-1}, B block tokens, N prefix
 * length, d head dimension, k budget.  Layouts (row-major, last index fastest):
 *   Q  [H_q][B][d]    Kc, Vc [H_kv][N][d]    Kb, Vb [H_kv][B][d]
 *
 * Parity pins (tests marked "not gpu"): brute force in NumPy on tiny inputs,
 * torch's scaled_dot_product_attention on concatenated keys, torch.topk as a
 * set, the invariants sum_j score[h][j] = 1 and "k = N sparse equals exact",
 * closed forms (equal keys, zero queries, one dominant key), a hand-computed
 * worked example.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double dot_d(const float *a, const float *b, int d) {
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += (double)a[c] * (double)b[c];
    return acc;
}

/*
 * Exact block attention of the all-[MASK] block (Algorithm 1, main stream,
 * "Attn(Q, K, V, C)"; Section 4, Phase 1).  Every query (g, q) attends to the
 * N cached keys of its KV head and to all B keys of its own block (no mask
 * inside the block, the token itself included), in one softmax.
 *   O [H_q][B][d]        attention output
 *   lse_prefix [H_q][B]  optional (may be NULL): natural-log sum-exp over the prefix keys only
 */
void oracle_exact_block_attn(const float *Q, const float *Kc, const float *Vc, const float *Kb, const float *Vb,
                             int H_q, int H_kv, int B, int d, int64_t N, double scale, double *O, double *lse_prefix) {
    const int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int row = 0; row < H_q * B; ++row) {
        const int g = row / B, h = g / G;
        const float *qv = Q + (size_t)row * d;
        const float *kc = Kc + (size_t)h * N * d, *vc = Vc + (size_t)h * N * d;
        const float *kb = Kb + (size_t)h * B * d, *vb = Vb + (size_t)h * B * d;
        double *s = (double *)malloc(sizeof(double) * (size_t)(N + B));
        double m = -INFINITY;
        for (int64_t j = 0; j < N; ++j) { s[j] = scale * dot_d(qv, kc + j * d, d); if (s[j] > m) m = s[j]; }
        if (lse_prefix) {
            double Lp = 0.0;
            for (int64_t j = 0; j < N; ++j) Lp += exp(s[j] - m);
            lse_prefix[row] = (N > 0) ? m + log(Lp) : -INFINITY;
        }
        for (int i = 0; i < B; ++i) { s[N + i] = scale * dot_d(qv, kb + (size_t)i * d, d); if (s[N + i] > m) m = s[N + i]; }
        double L = 0.0;
        for (int64_t j = 0; j < N + B; ++j) L += exp(s[j] - m);
        double *o = O + (size_t)row * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int64_t j = 0; j < N; ++j) { const double p = exp(s[j] - m) / L; for (int c = 0; c < d; ++c) o[c] += p * (double)vc[j * d + c]; }
        for (int i = 0; i < B; ++i) { const double p = exp(s[N + i] - m) / L; for (int c = 0; c < d; ++c) o[c] += p * (double)vb[(size_t)i * d + c]; }
        free(s);
    }
}

/*
 * Block score (Algorithm 1, select stream; Eq. 4, which instantiates the
 * per-block case of Eq. 2 with the exact attention probabilities):
 *   A[g][q][:] = softmax over the N PREFIX keys of Q[g][q] . Kc[h][:] / sqrt(d)
 *   score[h][j] = 1/(G B) * sum_{g in group(h)} sum_q A[g][q][j]
 * A is materialised per KV head as a (G*B) x N matrix, exactly as written.
 *   score [H_kv][N]
 */
void oracle_block_score(const float *Q, const float *Kc, int H_q, int H_kv, int B, int d, int64_t N, double scale,
                        double *score) {
    const int G = H_q / H_kv, M = G * B;
    if (N <= 0) return;
    double *A = (double *)malloc(sizeof(double) * (size_t)M * (size_t)N);
    for (int h = 0; h < H_kv; ++h) {
        const float *kc = Kc + (size_t)h * N * d;
#pragma omp parallel for schedule(dynamic, 1)
        for (int r = 0; r < M; ++r) {                       /* r = (g - hG) * B + q */
            const float *qv = Q + ((size_t)h * G * B + r) * d;
            double *a = A + (size_t)r * N;
            double m = -INFINITY, L = 0.0;
            for (int64_t j = 0; j < N; ++j) { a[j] = scale * dot_d(qv, kc + j * d, d); if (a[j] > m) m = a[j]; }
            for (int64_t j = 0; j < N; ++j) { a[j] = exp(a[j] - m); L += a[j]; }
            for (int64_t j = 0; j < N; ++j) a[j] /= L;
        }
#pragma omp parallel for schedule(static)
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int r = 0; r < M; ++r) acc += A[(size_t)r * N + j];
            score[(size_t)h * N + j] = acc / (double)M;
        }
    }
    free(A);
}

typedef struct { double s; int32_t j; } scored_t;
static int cmp_score_desc(const void *a, const void *b) {
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->j > y->j) - (x->j < y->j);                   /* equal scores: smaller position first */
}
static int cmp_i32(const void *a, const void *b) { int32_t x = *(const int32_t *)a, y = *(const int32_t *)b; return (x > y) - (x < y); }

/*
 * Top-k selection (Algorithm 1, "S <- Top-k(alpha)"): the k_eff = min(k, N)
 * positions with the largest score, by a full sort of all N entries; equal
 * scores are broken toward the smaller position.  idx [k] receives the
 * selected positions in ascending order, slots >= k_eff are set to -1.
 * Returns k_eff.
 */
int oracle_topk(const double *score, int64_t N, int k, int32_t *idx) {
    int k_eff = (int64_t)k < N ? k : (int)N;
    scored_t *v = (scored_t *)malloc(sizeof(scored_t) * (size_t)(N > 0 ? N : 1));
    for (int64_t j = 0; j < N; ++j) { v[j].s = score[j]; v[j].j = (int32_t)j; }
    qsort(v, (size_t)N, sizeof(scored_t), cmp_score_desc);
    for (int t = 0; t < k_eff; ++t) idx[t] = v[t].j;
    qsort(idx, (size_t)k_eff, sizeof(int32_t), cmp_i32);
    for (int t = k_eff; t < k; ++t) idx[t] = -1;
    free(v);
    return k_eff;
}

/*
 * Sparse reuse step (Algorithm 1, Phase 2, "SparseAttn(Q, K, V, C[S])"):
 * as the exact pass, but the prefix part of the softmax runs only over the
 * cache rows idx[h][0 .. k_eff-1]; the block's own B keys stay dense.
 *   idx [H_kv][k] int32, k_eff entries used per head
 */
void oracle_sparse_block_attn(const float *Q, const float *Kc, const float *Vc, const float *Kb, const float *Vb,
                              const int32_t *idx, int k, int k_eff, int H_q, int H_kv, int B, int d, int64_t N,
                              double scale, double *O) {
    const int G = H_q / H_kv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int row = 0; row < H_q * B; ++row) {
        const int g = row / B, h = g / G;
        const float *qv = Q + (size_t)row * d;
        const float *kc = Kc + (size_t)h * N * d, *vc = Vc + (size_t)h * N * d;
        const float *kb = Kb + (size_t)h * B * d, *vb = Vb + (size_t)h * B * d;
        const int32_t *sel = idx + (size_t)h * k;
        const int n = k_eff + B;
        double *s = (double *)malloc(sizeof(double) * (size_t)n);
        double m = -INFINITY;
        for (int t = 0; t < k_eff; ++t) { s[t] = scale * dot_d(qv, kc + (size_t)sel[t] * d, d); if (s[t] > m) m = s[t]; }
        for (int i = 0; i < B; ++i) { s[k_eff + i] = scale * dot_d(qv, kb + (size_t)i * d, d); if (s[k_eff + i] > m) m = s[k_eff + i]; }
        double L = 0.0;
        for (int t = 0; t < n; ++t) L += exp(s[t] - m);
        double *o = O + (size_t)row * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int t = 0; t < k_eff; ++t) { const double p = exp(s[t] - m) / L; for (int c = 0; c < d; ++c) o[c] += p * (double)vc[(size_t)sel[t] * d + c]; }
        for (int i = 0; i < B; ++i) { const double p = exp(s[k_eff + i] - m) / L; for (int c = 0; c < d; ++c) o[c] += p * (double)vb[(size_t)i * d + c]; }
        free(s);
    }
}

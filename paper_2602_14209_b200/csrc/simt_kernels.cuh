// Portable CUDA-core kernels for every stage of the path (fp32 FMA, no tensor cores).
// They accept every shape the ABI allows and serve as the safe path for shapes the
// tensor-core kernels do not cover, and as an on-device cross-check.
#pragma once
#include "common.cuh"

namespace mage {
namespace simt {

constexpr int kRows = 64;      // query rows per CTA tile
constexpr int kKeys = 64;      // keys per smem tile
constexpr int kThreads = 256;
constexpr int kPsLd = kKeys + 1;
constexpr size_t kSmemBytes = (size_t)(kD * kRows + kD * kKeys + kKeys * kD + kRows * kPsLd) * sizeof(float) + kKeys * sizeof(int);

enum class Mode { kExactPartial, kSparseFinal };

// Load 64 query rows of group h (rows r0 .. r0+63 of the M = G*B rows) transposed into Qs[c][r] as fp32.
__device__ __forceinline__ void load_q_tile(const KvView &kv, const __nv_bfloat16 *q, int p, int h, int r0, float *Qs) {
    const int t = threadIdx.x, row = t >> 2, quarter = t & 3, r = r0 + row;
    float vals[32];
    if (r < kv.M) {
        const __nv_bfloat16 *src = q + ((long long)(p * kv.H_q + h * kv.G) * kv.B + r) * kD + quarter * 32;
#pragma unroll
        for (int i = 0; i < 4; ++i) bf16x8_to_float(reinterpret_cast<const uint4 *>(src)[i], vals + 8 * i);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) vals[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) Qs[(quarter * 32 + i) * kRows + row] = vals[i];
}

// acc[i][c] = <Q row ty*4+i, K key tx*4+c> over d = 128 (raw dot product, fp32).
__device__ __forceinline__ void qk_tile(const float *Qs, const float *Ks, int ty, int tx, float acc[4][4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[i][c] = 0.f;
#pragma unroll 8
    for (int dd = 0; dd < kD; ++dd) {
        const float4 q4 = *reinterpret_cast<const float4 *>(Qs + dd * kRows + ty * 4);
        const float4 k4 = *reinterpret_cast<const float4 *>(Ks + dd * kKeys + tx * 4);
        const float qa[4] = {q4.x, q4.y, q4.z, q4.w}, ka[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[i][c] = fmaf(qa[i], ka[c], acc[i][c]);
    }
}

// Flash-style attention of a 64-row tile over a list of keys.
//  kExactPartial: keys are one chunk of the prefix (or, for chunk index n_chunks, the block's own B keys);
//                 writes the unnormalised partial (O, m, l) of the chunk to the workspace.
//  kSparseFinal : keys are the k_eff selected cache rows followed by the block's B keys; writes bf16 output.
template <Mode MODE>
__global__ void __launch_bounds__(kThreads) attn_kernel(KvView kv, Plan plan, const __nv_bfloat16 *__restrict__ q,
                                                        const __nv_bfloat16 *__restrict__ k_blk,
                                                        const __nv_bfloat16 *__restrict__ v_blk,
                                                        const int *__restrict__ indices, const int *__restrict__ k_eff_arr,
                                                        int k, float scale_log2, float *__restrict__ ws,
                                                        __nv_bfloat16 *__restrict__ out, unsigned *status) {
    extern __shared__ __align__(16) float smem[];
    float *Qs = smem, *Ks = Qs + kD * kRows, *Vs = Ks + kD * kKeys, *Ps = Vs + kKeys * kD;
    int *key_ok = reinterpret_cast<int *>(Ps + kRows * kPsLd);

    const int r0 = blockIdx.x * kRows, chunk = blockIdx.y, z = blockIdx.z, p = z / kv.H_kv, h = z % kv.H_kv;
    const int N = seq_len_of(kv, p);
    int n_cache, n_total, j_begin = 0;
    if (MODE == Mode::kExactPartial) {
        if (chunk < plan.n_chunks) {
            j_begin = chunk * plan.chunk_len;
            if (j_begin >= N) return;
            n_cache = min(plan.chunk_len, N - j_begin);
            n_total = n_cache;
        } else {
            n_cache = 0;
            n_total = kv.B;
        }
    } else {
        n_cache = min(max(k_eff_arr[p], 0), k);
        n_total = n_cache + kv.B;
    }
    const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
    load_q_tile(kv, q, p, h, r0, Qs);

    float m_run[4], l_run[4], o[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m_run[i] = -INFINITY;
        l_run[i] = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) o[i][c] = 0.f;
    }

    for (int t0 = 0; t0 < n_total; t0 += kKeys) {
        __syncthreads();   // previous tile fully consumed (also orders the Q tile store before its first use)
        {   // stage keys t0 .. t0+63: K transposed to Ks[c][key], V natural Vs[key][c]
            const int key = t >> 2, quarter = t & 3, tk = t0 + key;
            const __nv_bfloat16 *kp = nullptr, *vp = nullptr;
            if (tk < n_total) {
                if (tk < n_cache) {
                    int j = j_begin + tk;
                    bool ok = true;
                    if (MODE == Mode::kSparseFinal) {
                        j = indices[(long long)z * k + tk];
                        if (j < 0 || j >= N) { ok = false; if (status) atomicOr(status, MAGE_DEV_BAD_INDEX); }
                    }
                    if (ok) {
                        const long long off = cache_row_offset(kv, p, h, j, status);
                        if (off >= 0) { kp = kv.k + off; vp = kv.v + off; }
                    }
                } else {
                    const long long off = ((long long)z * kv.B + (tk - n_cache)) * kD;
                    kp = k_blk + off; vp = v_blk + off;
                }
            }
            float kvals[32], vvals[32];
            if (kp) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    bf16x8_to_float(reinterpret_cast<const uint4 *>(kp + quarter * 32)[i], kvals + 8 * i);
                    bf16x8_to_float(reinterpret_cast<const uint4 *>(vp + quarter * 32)[i], vvals + 8 * i);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) { kvals[i] = 0.f; vvals[i] = 0.f; }
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) Ks[(quarter * 32 + i) * kKeys + key] = kvals[i];
#pragma unroll
            for (int i = 0; i < 8; ++i) reinterpret_cast<float4 *>(Vs + key * kD + quarter * 32)[i] = reinterpret_cast<float4 *>(vvals)[i];
            if (quarter == 0) key_ok[key] = kp != nullptr;
        }
        __syncthreads();
        float s[4][4];
        qk_tile(Qs, Ks, ty, tx, s);
        bool ok[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) ok[c] = key_ok[tx * 4 + c] != 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) { s[i][c] = ok[c] ? s[i][c] * scale_log2 : -INFINITY; mx = fmaxf(mx, s[i][c]); }
#pragma unroll
            for (int w = 1; w < 16; w <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, w));
            const float m_new = fmaxf(m_run[i], mx);
            const float m_safe = m_new == -INFINITY ? 0.f : m_new;
            const float alpha = exp2f(m_run[i] - m_safe);       // m_run = -inf gives 0
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) { s[i][c] = exp2f(s[i][c] - m_safe); sum += s[i][c]; Ps[(ty * 4 + i) * kPsLd + tx * 4 + c] = s[i][c]; }
#pragma unroll
            for (int w = 1; w < 16; w <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, w);
            l_run[i] = l_run[i] * alpha + sum;
            m_run[i] = m_new;
#pragma unroll
            for (int c = 0; c < 8; ++c) o[i][c] *= alpha;
        }
        __syncthreads();
        for (int j = 0; j < kKeys; ++j) {
            const float4 va = *reinterpret_cast<const float4 *>(Vs + j * kD + tx * 4);
            const float4 vb = *reinterpret_cast<const float4 *>(Vs + j * kD + 64 + tx * 4);
            const float vv[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float pij = Ps[(ty * 4 + i) * kPsLd + j];
#pragma unroll
                for (int c = 0; c < 8; ++c) o[i][c] = fmaf(pij, vv[c], o[i][c]);
            }
        }
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty * 4 + i;
        if (r >= kv.M) continue;
        if (MODE == Mode::kExactPartial) {
            const size_t item = (size_t)z * (plan.n_chunks + 1) + chunk;
            float *po = ws + plan.off_part_o + (item * plan.Mw + r) * kD;
            *reinterpret_cast<float4 *>(po + tx * 4) = make_float4(o[i][0], o[i][1], o[i][2], o[i][3]);
            *reinterpret_cast<float4 *>(po + 64 + tx * 4) = make_float4(o[i][4], o[i][5], o[i][6], o[i][7]);
            if (tx == 0) {
                float *pml = ws + plan.off_part_ml + (item * plan.Mw + r) * 2;
                pml[0] = m_run[i];
                pml[1] = l_run[i];
            }
        } else {
            const float inv = 1.f / l_run[i];
            __nv_bfloat16 *po = out + ((long long)(p * kv.H_q + h * kv.G) * kv.B + r) * kD;
            __nv_bfloat162 a0 = __floats2bfloat162_rn(o[i][0] * inv, o[i][1] * inv), a1 = __floats2bfloat162_rn(o[i][2] * inv, o[i][3] * inv);
            __nv_bfloat162 b0 = __floats2bfloat162_rn(o[i][4] * inv, o[i][5] * inv), b1 = __floats2bfloat162_rn(o[i][6] * inv, o[i][7] * inv);
            *reinterpret_cast<uint2 *>(po + tx * 4) = make_uint2(*reinterpret_cast<unsigned *>(&a0), *reinterpret_cast<unsigned *>(&a1));
            *reinterpret_cast<uint2 *>(po + 64 + tx * 4) = make_uint2(*reinterpret_cast<unsigned *>(&b0), *reinterpret_cast<unsigned *>(&b1));
        }
    }
}

// Block score of 64 consecutive prefix positions of one KV head (Eq. 4), given each row's prefix log-sum-exp:
// score[j] = 1/M * sum_r exp2(s_rj * scale_log2 - lse2_r), summed over the M rows in a fixed order.
__global__ void __launch_bounds__(kThreads) score_kernel(KvView kv, Plan plan, const __nv_bfloat16 *__restrict__ q,
                                                         float scale_log2, const float *__restrict__ ws,
                                                         float *__restrict__ scores, unsigned *status) {
    extern __shared__ __align__(16) float smem[];
    float *Qs = smem, *Ks = Qs + kD * kRows, *red = Ks + kD * kKeys;   // red: [16][64]
    __shared__ int key_bad[kKeys];
    const int j0 = blockIdx.x * kKeys, z = blockIdx.z, p = z / kv.H_kv, h = z % kv.H_kv;
    const int N = seq_len_of(kv, p);
    if (j0 >= N) return;
    const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
    {
        const int key = t >> 2, quarter = t & 3, j = j0 + key;
        float kvals[32];
        long long off = -1;
        if (j < N) off = cache_row_offset(kv, p, h, j, status);
        if (quarter == 0) key_bad[key] = j < N && off < 0;    // page id out of range: the key is skipped, its score is 0
        if (off >= 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) bf16x8_to_float(reinterpret_cast<const uint4 *>(kv.k + off + quarter * 32)[i], kvals + 8 * i);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) kvals[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) Ks[(quarter * 32 + i) * kKeys + key] = kvals[i];
    }
    const float *neg_lse = ws + plan.off_neg_lse + (size_t)z * plan.Mw;
    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int r0 = 0; r0 < kv.M; r0 += kRows) {
        __syncthreads();
        load_q_tile(kv, q, p, h, r0, Qs);
        __syncthreads();
        float s[4][4];
        qk_tile(Qs, Ks, ty, tx, s);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + ty * 4 + i;
            if (r < kv.M) {
                const float nl = neg_lse[r];
#pragma unroll
                for (int c = 0; c < 4; ++c) col[c] += exp2f(fmaf(s[i][c], scale_log2, nl));
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 4; ++c) red[ty * kKeys + tx * 4 + c] = col[c];
    __syncthreads();
    if (t < kKeys && j0 + t < N) {
        float acc = 0.f;
        for (int y = 0; y < 16; ++y) acc += red[y * kKeys + t];
        scores[(size_t)z * kv.N_max + j0 + t] = key_bad[t] ? 0.f : acc / (float)kv.M;
    }
}

}  // namespace simt

// Merge the per-chunk partials of the exact pass: one warp per query row.
//  - log-sum-exp over the prefix chunks only -> neg_lse (log2 domain), used by the score kernels;
//  - prefix chunks + the block's own keys -> normalised bf16 output.
__global__ void __launch_bounds__(128) combine_kernel(KvView kv, Plan plan, float *__restrict__ ws,
                                                      __nv_bfloat16 *__restrict__ out, int lse_only) {
    // may have been launched while the attention kernel was still running (programmatic dependent launch): wait for it,
    // then let the score kernel's CTAs be scheduled
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int rows_total = kv.P * kv.H_kv * kv.M;
    if (warp >= rows_total) return;
    const int z = warp / kv.M, r = warp % kv.M, p = z / kv.H_kv, h = z % kv.H_kv;
    const int N = seq_len_of(kv, p);
    const int nc = (N + plan.chunk_len - 1) / plan.chunk_len;
    const size_t item0 = (size_t)z * (plan.n_chunks + 1);
    const float *ml = ws + plan.off_part_ml;
    const float *po = ws + plan.off_part_o;
    // Lane c % 32 owns chunk c's (m, l): all of them are loaded at once (up to kMaxPerLane per lane), the maximum and the
    // sum are warp reductions in a fixed order, and the weights then travel by shuffle -- no chain of dependent loads.
    constexpr int kMaxPerLane = 5;                       // 148 chunks per head at most
    float m_c[kMaxPerLane], l_c[kMaxPerLane];
    float m_pre = -INFINITY;
#pragma unroll
    for (int u = 0; u < kMaxPerLane; ++u) {
        const int c = lane + 32 * u;
        m_c[u] = -INFINITY;
        l_c[u] = 0.f;
        if (c < nc) {
            const float2 e = *reinterpret_cast<const float2 *>(ml + ((item0 + c) * plan.Mw + r) * 2);
            m_c[u] = e.x;
            l_c[u] = e.y;
        }
        m_pre = fmaxf(m_pre, m_c[u]);
    }
#pragma unroll
    for (int w = 16; w; w >>= 1) m_pre = fmaxf(m_pre, __shfl_xor_sync(0xffffffffu, m_pre, w));
    float l_pre = 0.f;
#pragma unroll
    for (int u = 0; u < kMaxPerLane; ++u) l_pre += (lane + 32 * u < nc) ? l_c[u] * exp2f(m_c[u] - m_pre) : 0.f;
#pragma unroll
    for (int w = 16; w; w >>= 1) l_pre += __shfl_xor_sync(0xffffffffu, l_pre, w);
    if (lane == 0) ws[plan.off_neg_lse + (size_t)z * plan.Mw + r] = nc > 0 ? -(m_pre + log2f(l_pre)) : 0.f;
    if (lse_only) return;                                 // the select stream's own pass: no block chunk, no output
    const float *eb = ml + ((item0 + plan.n_chunks) * plan.Mw + r) * 2;
    const float m_blk = eb[0], l_blk = eb[1];
    const float m_all = fmaxf(m_pre, m_blk);
    const float w_blk = exp2f(m_blk - m_all);
    const float l_all = l_blk * w_blk + (nc > 0 ? l_pre * exp2f(m_pre - m_all) : 0.f);
    float w_c[kMaxPerLane];
#pragma unroll
    for (int u = 0; u < kMaxPerLane; ++u) w_c[u] = (lane + 32 * u < nc) ? exp2f(m_c[u] - m_all) : 0.f;
    float4 acc = *reinterpret_cast<const float4 *>(po + ((item0 + plan.n_chunks) * plan.Mw + r) * kD + lane * 4);
    acc.x *= w_blk; acc.y *= w_blk; acc.z *= w_blk; acc.w *= w_blk;
#pragma unroll
    for (int u = 0; u < kMaxPerLane; ++u) {
        if (32 * u >= nc) break;
        const int n_here = min(32, nc - 32 * u);
        for (int c0 = 0; c0 < n_here; c0 += 4) {         // four independent 16-byte loads in flight per lane
            float4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q)
                v[q] = c0 + q < n_here ? *reinterpret_cast<const float4 *>(po + ((item0 + 32 * u + c0 + q) * plan.Mw + r) * kD + lane * 4)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int q = 0; q < 4; ++q) {                // chunks in ascending order: the result does not depend on timing
                const float w = __shfl_sync(0xffffffffu, w_c[u], (c0 + q) & 31);
                acc.x = fmaf(v[q].x, w, acc.x); acc.y = fmaf(v[q].y, w, acc.y); acc.z = fmaf(v[q].z, w, acc.z); acc.w = fmaf(v[q].w, w, acc.w);
            }
        }
    }
    const float inv = 1.f / l_all;
    __nv_bfloat16 *dst = out + ((long long)(p * kv.H_q + h * kv.G) * kv.B + r) * kD + lane * 4;
    __nv_bfloat162 a = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), b = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<unsigned *>(&a), *reinterpret_cast<unsigned *>(&b));
}

// Cache append (Algorithm 1, "C <- C || KV(x)"): one warp per (problem, KV head, block token) copies the 256-byte
// K row and V row to logical position N_p + token.  seq_lens is bumped by a second launch, after every row has
// read the old length.
__global__ void __launch_bounds__(128) append_rows_kernel(KvView kv, const __nv_bfloat16 *__restrict__ k_blk,
                                                          const __nv_bfloat16 *__restrict__ v_blk, const int *__restrict__ seq_lens,
                                                          unsigned *status) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int total = kv.P * kv.H_kv * kv.B;
    if (warp >= total) return;
    const int t = warp % kv.B, z = warp / kv.B, p = z / kv.H_kv, h = z % kv.H_kv;
    const int n = seq_lens[p];
    if (n < 0 || n + kv.B > kv.N_max) {
        if (status && lane == 0) atomicOr(status, MAGE_DEV_CACHE_FULL);
        return;
    }
    // every page the block touches must be mapped, or nothing of the block is written
    if (kv.page_size) {
        for (int j = n; j < n + kv.B; j += kv.page_size - (j % kv.page_size)) {
            const int page = kv.block_table[(long long)p * kv.max_pages + j / kv.page_size];
            if (page < 0 || page >= kv.num_pages) {
                if (status && lane == 0) atomicOr(status, MAGE_DEV_BAD_PAGE);
                return;
            }
        }
    }
    const long long off = cache_row_offset(kv, p, h, n + t, nullptr);
    if (off < 0) return;
    if (lane < 16) {
        const uint4 kx = reinterpret_cast<const uint4 *>(k_blk + (long long)warp * kD)[lane];
        const uint4 vx = reinterpret_cast<const uint4 *>(v_blk + (long long)warp * kD)[lane];
        reinterpret_cast<uint4 *>(const_cast<__nv_bfloat16 *>(kv.k) + off)[lane] = kx;
        reinterpret_cast<uint4 *>(const_cast<__nv_bfloat16 *>(kv.v) + off)[lane] = vx;
    }
}

__global__ void bump_seq_lens_kernel(KvView kv, int *seq_lens) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= kv.P) return;
    const int n = seq_lens[p];
    if (n < 0 || n + kv.B > kv.N_max) return;
    if (kv.page_size) {
        for (int j = n; j < n + kv.B; j += kv.page_size - (j % kv.page_size)) {
            const int page = kv.block_table[(long long)p * kv.max_pages + j / kv.page_size];
            if (page < 0 || page >= kv.num_pages) return;
        }
    }
    seq_lens[p] = n + kv.B;
}

}  // namespace mage

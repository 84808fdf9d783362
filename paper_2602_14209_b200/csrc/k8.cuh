// Keys and queries in 8 bits (e4m3) for the exact pass, the score pass and the reuse step.  The paper leaves cache
// compression to future work (Limitations), so the variant is defined here:
//
//   scale   one per (problem, KV head):  s = amax / 448 in single precision (1 when amax = 0); amax = largest |x| over the
//           head's rows -- the cached keys below seq_len for s_k, the G*B query rows of the call for s_q
//   code    cvt.rn.satfinite.e4m3( x / s ), the division in IEEE single precision: round to nearest even onto the e4m3
//           grid, magnitudes beyond 448 clamp to 448
//   keys    cache keys and the block's own keys both use the head's s_k (block keys larger than the cache's amax clamp)
//   logits  s_q s_k * (code_q . code_k): the products of two e4m3 numbers are exact in the tensor core's fp32 accumulation,
//           and s_q s_k is folded into the softmax scale of the head.  Values stay bf16.
//
// The codes of the cache are written once (and again for appended rows); queries and block keys are coded at every call.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mage {
namespace k8 {

constexpr float kE4m3Max = 448.f;

__device__ __forceinline__ unsigned short e4m3x2(float lo, float hi) {      // low byte = code of lo
    unsigned short r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float scale_of(float amax) { return amax > 0.f ? __fdiv_rn(amax, kE4m3Max) : 1.f; }

// 16 consecutive bf16 -> 16 codes
__device__ __forceinline__ uint4 code16(const uint4 &a, const uint4 &b, float s) {
    float x[16];
    bf16x8_to_float(a, x);
    bf16x8_to_float(b, x + 8);
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const unsigned lo = e4m3x2(__fdiv_rn(x[4 * i], s), __fdiv_rn(x[4 * i + 1], s));
        const unsigned hi = e4m3x2(__fdiv_rn(x[4 * i + 2], s), __fdiv_rn(x[4 * i + 3], s));
        w[i] = lo | (hi << 16);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ float amax8(const uint4 &a, float m) {
    float x[8];
    bf16x8_to_float(a, x);
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(x[i]));       // fmaxf drops a NaN operand
    return m;
}

constexpr int kRowsPerCta = 1024;

// Largest |key| per (problem, KV head) over rows [row_begin, seq_len): bit pattern of a non-negative float, merged with
// atomicMax (such patterns order like the numbers).  amax_bits must be zero on entry.
__global__ void __launch_bounds__(256) cache_amax_kernel(KvView kv, int row_begin, unsigned *amax_bits, unsigned *status) {
    const int z = blockIdx.y, p = z / kv.H_kv, h = z % kv.H_kv, N = seq_len_of(kv, p);
    const int r0 = row_begin + blockIdx.x * kRowsPerCta, r1 = min(N, r0 + kRowsPerCta);
    float m = 0.f;
    for (int j = r0 + (threadIdx.x >> 4); j < r1; j += 16) {
        const long long off = cache_row_offset(kv, p, h, j, status);
        if (off < 0) continue;
        m = amax8(*reinterpret_cast<const uint4 *>(kv.k + off + (threadIdx.x & 15) * 8), m);
    }
#pragma unroll
    for (int w = 16; w; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
    if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(amax_bits + z, __float_as_uint(m));
}
// in place: amax -> scale
__global__ void amax_to_scale_kernel(float *scale, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) scale[i] = scale_of(scale[i]);
}
// Codes of cache rows [row_begin, seq_len) under the head's scale; the code of element e of a row sits at the same
// element offset in k8 as the element itself in the key cache.
__global__ void __launch_bounds__(256) cache_code_kernel(KvView kv, int row_begin, const float *__restrict__ k_scale,
                                                         uint8_t *__restrict__ k8, unsigned *status) {
    const int z = blockIdx.y, p = z / kv.H_kv, h = z % kv.H_kv, N = seq_len_of(kv, p);
    const int r0 = row_begin + blockIdx.x * kRowsPerCta, r1 = min(N, r0 + kRowsPerCta);
    const float s = k_scale[z];
    const int piece = threadIdx.x & 7;                           // 16 elements of the row
    for (int j = r0 + (threadIdx.x >> 3); j < r1; j += 32) {
        const long long off = cache_row_offset(kv, p, h, j, status);
        if (off < 0) continue;
        const uint4 *src = reinterpret_cast<const uint4 *>(kv.k + off + piece * 16);
        *reinterpret_cast<uint4 *>(k8 + off + piece * 16) = code16(src[0], src[1], s);
    }
}

// One CTA per (problem, KV head): s_q from the head's G*B query rows, their codes, the codes of the block's own keys under
// s_k, and the head's factor s_q s_k for the kernels that follow.
__global__ void __launch_bounds__(256) block_code_kernel(KvView kv, const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_blk,
                                                         const float *__restrict__ k_scale, uint8_t *__restrict__ q8,
                                                         uint8_t *__restrict__ kb8, float *__restrict__ qk_scale) {
    __shared__ float red[8];
    ptx::pdl_wait();                 // launched with programmatic serialization: nothing is read before the predecessor is done
    ptx::pdl_launch_dependents();    // the pass that follows may set itself up meanwhile; it waits for this grid's end before reading
    const int z = blockIdx.x, p = z / kv.H_kv, h = z % kv.H_kv, tid = threadIdx.x;
    const size_t q_off = ((size_t)(p * kv.H_q + h * kv.G) * kv.B) * kD;
    const uint4 *qv = reinterpret_cast<const uint4 *>(q + q_off);
    const int n_q16 = kv.M * (kD / 16);                          // 16-element pieces of the head's queries
    // up to 256 rows stay in registers between the two passes (eight pieces per thread); longer heads are read again
    uint4 keep[16];
    float m = 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int j = tid + u * 256;
        if (j < n_q16) {
            keep[2 * u] = qv[2 * j];
            keep[2 * u + 1] = qv[2 * j + 1];
            m = amax8(keep[2 * u + 1], amax8(keep[2 * u], m));
        }
    }
    for (int j = tid + 2048; j < n_q16; j += 256) m = amax8(qv[2 * j + 1], amax8(qv[2 * j], m));
    const uint4 *bv = reinterpret_cast<const uint4 *>(k_blk + (size_t)z * kv.B * kD);
    uint4 kb0 = make_uint4(0, 0, 0, 0), kb1 = kb0, kb2 = kb0, kb3 = kb0;      // the block's keys: B <= 64 rows, two pieces per thread
    const int n_b16 = kv.B * (kD / 16);
    if (tid < n_b16) { kb0 = bv[2 * tid]; kb1 = bv[2 * tid + 1]; }
    if (tid + 256 < n_b16) { kb2 = bv[2 * (tid + 256)]; kb3 = bv[2 * (tid + 256) + 1]; }
#pragma unroll
    for (int w = 16; w; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
    if ((tid & 31) == 0) red[tid >> 5] = m;
    __syncthreads();
    m = red[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]);
    const float s_q = scale_of(m), s_k = k_scale[z];
    if (tid == 0) qk_scale[z] = s_q * s_k;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int j = tid + u * 256;
        if (j < n_q16) *reinterpret_cast<uint4 *>(q8 + q_off + (size_t)j * 16) = code16(keep[2 * u], keep[2 * u + 1], s_q);
    }
    for (int j = tid + 2048; j < n_q16; j += 256)
        *reinterpret_cast<uint4 *>(q8 + q_off + (size_t)j * 16) = code16(qv[2 * j], qv[2 * j + 1], s_q);
    const size_t b_off = (size_t)z * kv.B * kD;
    if (tid < n_b16) *reinterpret_cast<uint4 *>(kb8 + b_off + (size_t)tid * 16) = code16(kb0, kb1, s_k);
    if (tid + 256 < n_b16) *reinterpret_cast<uint4 *>(kb8 + b_off + (size_t)(tid + 256) * 16) = code16(kb2, kb3, s_k);
}

}  // namespace k8
}  // namespace mage

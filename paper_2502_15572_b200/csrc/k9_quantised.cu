// K9 -- quantised candidate search.  The paper does not search its datastore exactly: it
// hands the query to an approximate nearest-neighbour library (Section 3.5) whose core
// device is scoring against a compressed copy of the keys.  The equivalent here, with every
// step defined exactly so that it can be checked against a CPU statement of the same rules:
//
//   k8_ij = e4m3(256 k_ij)                       8-bit keys: half the bytes of a 16-bit store
//   h1_j  = e4m3(256 q_j),  h2_j = e4m3(16 (256 q_j - h1_j))       two-term 8-bit query
//   a_i   = sum_j (h1_j + h2_j / 16) k8_ij       approximate score (x 65536), on the tensor
//                                                cores (kind::f8f6f4) by the scan kernel
//   the m best a_i are scored exactly against the 16-bit keys and the n best are returned.
//
// E4M3: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits, largest finite value 448, no
// infinities; conversions round to nearest even and saturate.
//
// This file holds the three small kernels around the scan: the key quantiser (HBM-bound, run
// once per datastore), the query splitter, and the exact re-ranking with the value lookup.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

__device__ __forceinline__ uint32_t to_e4m3(float x)
{
    return (uint32_t)__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
}
__device__ __forceinline__ float from_e4m3(uint32_t c)
{
    const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)c, __NV_E4M3);
    return __half2float(*reinterpret_cast<const __half *>(&h));
}

template <typename T> __device__ __forceinline__ void unpack16(const uint4 &v, float *x);
template <> __device__ __forceinline__ void unpack16<__half>(const uint4 &v, float *x)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4 &v, float *x)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// 16 keys elements (two 16-byte loads) -> 16 codes (one 16-byte store) per thread and step.
template <typename T>
__global__ void __launch_bounds__(256) quantise_keys_kernel(const T *__restrict__ keys, long long total16,
                                                            uint4 *__restrict__ out)
{
    const uint4 *in = reinterpret_cast<const uint4 *>(keys);
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total16;
         i += (long long)gridDim.x * blockDim.x) {
        const uint4 a = __ldcs(in + 2 * i), b = __ldcs(in + 2 * i + 1);
        float x[16];
        unpack16<T>(a, x);
        unpack16<T>(b, x + 8);
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            w[k] = to_e4m3(256.f * x[4 * k]) | (to_e4m3(256.f * x[4 * k + 1]) << 8) |
                   (to_e4m3(256.f * x[4 * k + 2]) << 16) | (to_e4m3(256.f * x[4 * k + 3]) << 24);
        __stcs(out + i, make_uint4(w[0], w[1], w[2], w[3]));
    }
}

// One CTA per operand query: rows 2b (h1) and 2b+1 (h2) of the 8-bit operand, zero-padded to
// dpad8 bytes; queries past B are zero rows.  pack2 (d = 64, dpad8 = 128: two keys per store
// row): rows 4b .. 4b+3 = (h1|0), (h2|0), (0|h1), (0|h2).
__global__ void split_queries_e4m3_kernel(const float *__restrict__ qhat, int B, int d, uint8_t *__restrict__ qsplit8,
                                          int dpad8, int pack2)
{
    const int b = blockIdx.x;
    if (pack2) {
        uint8_t *r0 = qsplit8 + (size_t)(4 * b) * dpad8;
        for (int j = threadIdx.x; j < 64; j += blockDim.x) {
            uint32_t c1 = 0u, c2 = 0u;
            if (b < B) {
                const float q256 = 256.f * qhat[(size_t)b * d + j];
                c1 = to_e4m3(q256);
                c2 = to_e4m3(16.f * (q256 - from_e4m3(c1)));
            }
            r0[j] = (uint8_t)c1;
            r0[64 + j] = 0;
            r0[dpad8 + j] = (uint8_t)c2;
            r0[dpad8 + 64 + j] = 0;
            r0[2 * dpad8 + j] = 0;
            r0[2 * dpad8 + 64 + j] = (uint8_t)c1;
            r0[3 * dpad8 + j] = 0;
            r0[3 * dpad8 + 64 + j] = (uint8_t)c2;
        }
        return;
    }
    uint8_t *h1 = qsplit8 + (size_t)(2 * b) * dpad8, *h2 = h1 + dpad8;
    for (int j = threadIdx.x; j < dpad8; j += blockDim.x) {
        uint32_t c1 = 0u, c2 = 0u;
        if (b < B && j < d) {
            const float q256 = 256.f * qhat[(size_t)b * d + j];
            c1 = to_e4m3(q256);
            c2 = to_e4m3(16.f * (q256 - from_e4m3(c1)));
        }
        h1[j] = (uint8_t)c1;
        h2[j] = (uint8_t)c2;
    }
}

// Exact re-ranking: one CTA per query, a warp per candidate.  s = sum_j q_j k_ij in fp32 (the
// 16-bit key element converts exactly; four partial sums per lane, fixed reduction order),
// then the m candidates are sorted by (score descending, row ascending), the n best written
// out and their stored tokens copied (Section 3.5, f_D: k -> v).
template <typename T>
__global__ void __launch_bounds__(256) rerank_kernel(const T *__restrict__ keys, int d, long long N,
                                                     const float *__restrict__ qhat, const int32_t *__restrict__ cand,
                                                     int m, int top_n, long long extra_id,
                                                     const int32_t *__restrict__ next_tokens,
                                                     int stored_len, int draft_len, int32_t *__restrict__ out_ids,
                                                     float *__restrict__ out_scores, int32_t *__restrict__ out_tokens)
{
    __shared__ unsigned long long packed[kListLen + 1];
    __shared__ int win[kListLen];
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float *q = qhat + (size_t)b * d;
    // slot kListLen: one extra candidate (the last key of an odd-sized packed store), never a duplicate
    for (int r = warp; r <= kListLen; r += 8) {
        const long long id = r < m ? cand[(size_t)b * m + r] : r == kListLen ? extra_id : -1;
        unsigned long long p = 0ull;
        if (id >= 0 && id < N) {                             // warp-uniform
            const uint4 *row = reinterpret_cast<const uint4 *>(keys + (size_t)id * d);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            for (int c = lane; c < d / 8; c += 32) {          // d is a multiple of 16
                float x[8];
                unpack16<T>(__ldg(row + c), x);
                const float4 q0 = *reinterpret_cast<const float4 *>(q + 8 * c);
                const float4 q1 = *reinterpret_cast<const float4 *>(q + 8 * c + 4);
                a0 = fmaf(q0.x, x[0], a0); a1 = fmaf(q0.y, x[1], a1); a2 = fmaf(q0.z, x[2], a2); a3 = fmaf(q0.w, x[3], a3);
                a0 = fmaf(q1.x, x[4], a0); a1 = fmaf(q1.y, x[5], a1); a2 = fmaf(q1.z, x[6], a2); a3 = fmaf(q1.w, x[7], a3);
            }
            float s = (a0 + a1) + (a2 + a3);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
            p = pack_candidate(s, (uint32_t)id);
        }
        if (lane == 0) packed[r] = p;
    }
    __syncthreads();
    if (warp == 0) {
        unsigned long long x = warp_sort_desc(packed[lane], lane);
        x = warp_merge_top32(x, lane == 0 ? packed[kListLen] : 0ull, lane);      // a sorted list of one
        if (lane < top_n) {
            const int id = x ? (int32_t)candidate_id(x) : -1;
            out_ids[(size_t)b * top_n + lane] = id;
            out_scores[(size_t)b * top_n + lane] = x ? candidate_score(x) : -INFINITY;
            win[lane] = id;
        }
    }
    __syncthreads();
    const int total = top_n * draft_len;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int r = i / draft_len, t = i - r * draft_len;
        const long long id = win[r];
        out_tokens[(size_t)b * total + i] = (id >= 0 && id < N) ? next_tokens[(size_t)id * stored_len + t] : -1;
    }
}

}  // namespace

cudaError_t launch_quantise_keys(const void *keys, int dtype, long long N, int d, void *out_q8, int sms,
                                 cudaStream_t stream)
{
    const long long total16 = N * (long long)d / 16;          // d is a multiple of 16
    if (total16 <= 0) return cudaSuccess;
    long long blocks = (total16 + 255) / 256;
    if (blocks > (long long)sms * 16) blocks = (long long)sms * 16;
    if (dtype == kF16)
        quantise_keys_kernel<__half><<<(int)blocks, 256, 0, stream>>>(static_cast<const __half *>(keys), total16,
                                                                       static_cast<uint4 *>(out_q8));
    else
        quantise_keys_kernel<__nv_bfloat16><<<(int)blocks, 256, 0, stream>>>(
            static_cast<const __nv_bfloat16 *>(keys), total16, static_cast<uint4 *>(out_q8));
    return cudaGetLastError();
}

cudaError_t launch_split_queries_e4m3(const float *qhat, int B, int rows, int d, void *qsplit8, int dpad8,
                                      int pack2, cudaStream_t stream)
{
    split_queries_e4m3_kernel<<<rows, 256, 0, stream>>>(qhat, B, d, static_cast<uint8_t *>(qsplit8), dpad8, pack2);
    return cudaGetLastError();
}

cudaError_t launch_rerank(const void *keys, int dtype, int d, long long N, const float *qhat, const int32_t *cand,
                          int B, int m, int top_n, long long extra_id, const int32_t *next_tokens, int stored_len,
                          int draft_len, int32_t *out_ids, float *out_scores, int32_t *out_tokens,
                          cudaStream_t stream)
{
    if (dtype == kF16)
        rerank_kernel<__half><<<B, 256, 0, stream>>>(static_cast<const __half *>(keys), d, N, qhat, cand, m, top_n,
                                                      extra_id, next_tokens, stored_len, draft_len, out_ids, out_scores,
                                                      out_tokens);
    else
        rerank_kernel<__nv_bfloat16><<<B, 256, 0, stream>>>(static_cast<const __nv_bfloat16 *>(keys), d, N, qhat,
                                                            cand, m, top_n, extra_id, next_tokens, stored_len, draft_len,
                                                            out_ids, out_scores, out_tokens);
    return cudaGetLastError();
}

}  // namespace dresd

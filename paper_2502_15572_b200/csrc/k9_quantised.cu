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
// This file holds the kernels around the scan: the key quantiser (HBM-bound, run once per
// datastore) and the exact re-ranking with the value lookup; the query terms are written by
// the preprocessing kernel.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

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

// Grid merge of the approximate lists + exact re-ranking + value lookup, one CTA (16 warps) per
// query.  The per-CTA lists (sorted by approximate score, m entries each) are folded as in the
// exact path; the m survivors are then scored exactly, a warp per candidate: s = sum_j q_j k_ij
// in fp32 (the 16-bit key element converts exactly; four partial sums per lane, fixed reduction
// order); the candidates are sorted by (score descending, row ascending), the n best written
// out and their stored tokens copied (Section 3.5, f_D: k -> v).  extra_id >= 0 is one more
// candidate for every query (the last key of an odd-sized packed store).
constexpr int kRerankWarps = 16;

template <typename T>
__global__ void __launch_bounds__(kRerankWarps * 32)
merge_rerank_kernel(const unsigned long long *__restrict__ cand, int lists, int B, const T *__restrict__ keys, int d,
                    long long N, const float *__restrict__ qhat, int mcand, int top_n, long long extra_id,
                    const int32_t *__restrict__ want_first, const int32_t *__restrict__ next_tokens, int stored_len, int draft_len,
                    int32_t *__restrict__ out_ids, float *__restrict__ out_scores, int32_t *__restrict__ out_tokens)
{
    __shared__ unsigned long long part[kRerankWarps][kListLen];
    __shared__ unsigned long long packed[kListLen + 1];
    __shared__ int win[kListLen];
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_wait();                           // the scan's lists are complete and visible
    pdl_launch_dependents();

    unsigned long long m = 0ull;
    // eight lists in flight per warp before the dependent merge chain; empty lists (CTAs that saw
    // no candidate: short scans, token windows) are skipped
    for (int g0 = warp; g0 < lists; g0 += 8 * kRerankWarps) {
        unsigned long long l[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int g = g0 + k * kRerankWarps;
            l[k] = g < lists ? cand[((size_t)g * B + b) * kCandStride + lane] : 0ull;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (shfl_u64(l[k], 0) != 0ull) m = warp_merge_top32(m, l[k], lane);      // sorted: slot 0 is the best
    }
    part[warp][lane] = m;
    __syncthreads();
    for (int span = kRerankWarps / 2; span >= 1; span >>= 1) {
        if (warp < span) {
            m = warp_merge_top32(part[warp][lane], part[warp + span][lane], lane);
            part[warp][lane] = m;
        }
        __syncthreads();
    }
    // part[0]: the best approximate scores with their rows; the first mcand of them are the candidates
    const float *q = qhat + (size_t)b * d;
    for (int r = warp; r <= kListLen; r += kRerankWarps) {
        const unsigned long long c = r < mcand ? part[0][r] : 0ull;       // exactly the m best, as defined
        long long id = r < kListLen ? (c ? (long long)candidate_id(c) : -1) : extra_id;
        // the extra candidate did not pass the scan's first-token test: apply it here
        if (r == kListLen && id >= 0 && want_first && want_first[b] >= 0 &&
            next_tokens[(size_t)id * stored_len] != want_first[b])
            id = -1;
        unsigned long long p = 0ull;
        if (id >= 0 && id < N) {                             // warp-uniform
            const uint4 *row = reinterpret_cast<const uint4 *>(keys + (size_t)id * d);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            for (int cc = lane; cc < d / 8; cc += 32) {       // d is a multiple of 16
                float x[8];
                unpack16<T>(__ldg(row + cc), x);
                const float4 q0 = *reinterpret_cast<const float4 *>(q + 8 * cc);
                const float4 q1 = *reinterpret_cast<const float4 *>(q + 8 * cc + 4);
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

cudaError_t launch_merge_rerank(const unsigned long long *cand, int lists, int B, const void *keys, int dtype, int d,
                                long long N, const float *qhat, int mcand, int top_n, long long extra_id,
                                const int32_t *want_first, const int32_t *next_tokens, int stored_len, int draft_len,
                                int32_t *out_ids, float *out_scores, int32_t *out_tokens, cudaStream_t stream)
{
    if (dtype == kF16)
        return launch_dependent(merge_rerank_kernel<__half>, dim3(B), dim3(kRerankWarps * 32), 0, stream, cand, lists, B,
                                static_cast<const __half *>(keys), d, N, qhat, mcand, top_n, extra_id, want_first,
                                next_tokens, stored_len, draft_len, out_ids, out_scores, out_tokens);
    return launch_dependent(merge_rerank_kernel<__nv_bfloat16>, dim3(B), dim3(kRerankWarps * 32), 0, stream, cand, lists,
                            B, static_cast<const __nv_bfloat16 *>(keys), d, N, qhat, mcand, top_n, extra_id, want_first,
                            next_tokens, stored_len, draft_len, out_ids, out_scores, out_tokens);
}

}  // namespace dresd

// Token-level half of batch verification (Section 3.6 of the paper) that needs no LLM:
//   K6a  prepare: the n retrieved continuations of a query become the n x L draft
//        matrix that is sent for verification -- everything after the first EOS is EOS
//        (Fig. 3: the EOS id is the padding), missing neighbours are all-EOS and
//        invalid, and a draft equal to a better-ranked one is marked invalid;
//   K6b  accept: given the LLM's own token at every draft position, the longest draft
//        prefix that matches exactly is accepted, followed by the LLM's token at the
//        first mismatch (so that every iteration yields at least one token, Section 3.1).
// One warp per query, one lane per draft (n <= 32).
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

__global__ void drafts_prepare_kernel(const int32_t *__restrict__ tokens, const int32_t *__restrict__ ids,
                                      int n, int L, int eos, int32_t *__restrict__ drafts,
                                      int32_t *__restrict__ valid)
{
    const int b = blockIdx.x, r = threadIdx.x;
    extern __shared__ int32_t sm[];                      // [n][L] padded drafts
    if (r < n) {
        const bool present = ids[(size_t)b * n + r] >= 0;
        bool ended = !present;
        for (int t = 0; t < L; ++t) {
            int32_t x = ended ? eos : tokens[((size_t)b * n + r) * L + t];
            sm[r * L + t] = x;
            drafts[((size_t)b * n + r) * L + t] = x;
            ended |= x == eos;
        }
    }
    __syncthreads();
    if (r < n) {
        bool ok = ids[(size_t)b * n + r] >= 0;
        for (int p = 0; p < r && ok; ++p) {               // equal to a better-ranked draft?
            if (ids[(size_t)b * n + p] < 0) continue;
            bool same = true;
            for (int t = 0; t < L && same; ++t) same = sm[p * L + t] == sm[r * L + t];
            ok = !same;
        }
        valid[(size_t)b * n + r] = ok ? 1 : 0;
    }
}

__global__ void drafts_accept_kernel(const int32_t *__restrict__ drafts, const int32_t *__restrict__ valid,
                                     const int32_t *__restrict__ llm, int n, int L,
                                     int32_t *__restrict__ out_best, int32_t *__restrict__ out_len,
                                     int32_t *__restrict__ out_tokens)
{
    const int b = blockIdx.x, lane = threadIdx.x;
    int a = -1;                                           // matched prefix length of this lane's draft
    if (lane < n && valid[(size_t)b * n + lane]) {
        a = 0;
        while (a < L && drafts[((size_t)b * n + lane) * L + a] == llm[((size_t)b * n + lane) * (L + 1) + a]) ++a;
    }
    // longest match wins, ties to the better-ranked (lower) draft
    int key = a >= 0 ? (a << 6) | (63 - lane) : -1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xFFFFFFFFu, key, o));
    const int best = key >= 0 ? 63 - (key & 63) : -1;
    const int len = key >= 0 ? key >> 6 : 0;
    if (lane == 0) {
        out_best[b] = best;
        out_len[b] = len + 1;
    }
    const int src = best >= 0 ? best : 0;                 // with no valid draft: the LLM's own next token
    for (int t = lane; t <= L; t += 32) {
        int32_t x = -1;
        if (t < len) x = drafts[((size_t)b * n + src) * L + t];
        else if (t == len) x = llm[((size_t)b * n + src) * (L + 1) + t];
        out_tokens[(size_t)b * (L + 1) + t] = x;
    }
}

}  // namespace

cudaError_t launch_drafts_prepare(const int32_t *tokens, const int32_t *ids, int B, int n, int L, int eos,
                                  int32_t *drafts, int32_t *valid, cudaStream_t stream)
{
    drafts_prepare_kernel<<<B, 32, sizeof(int32_t) * (size_t)n * L, stream>>>(tokens, ids, n, L, eos, drafts, valid);
    return cudaGetLastError();
}

cudaError_t launch_drafts_accept(const int32_t *drafts, const int32_t *valid, const int32_t *llm, int B, int n,
                                 int L, int32_t *out_best, int32_t *out_len, int32_t *out_tokens,
                                 cudaStream_t stream)
{
    drafts_accept_kernel<<<B, 32, 0, stream>>>(drafts, valid, llm, n, L, out_best, out_len, out_tokens);
    return cudaGetLastError();
}

}  // namespace dresd

// ---------------------------------------------------------------------------------
// Row-sharded datastore: the exchange step.  Every shard (GPU) returns its own top-n
// with LOCAL row ids; the top-n of the union is the top-n of the whole datastore
// (Eq. 3 is an arg max over D, and D is the disjoint union of the shards).  One warp
// per query folds the P sorted lists with the same bitonic merges as the grid merge,
// on global ids (local id + the shard's row offset), then copies the winners' tokens.
// ---------------------------------------------------------------------------------
namespace dresd {
namespace {

// stride_x: distance in elements between two shards' blocks of array x (dense arrays: B n and
// B n L; results packed per shard for a single all-gather: the packed block size for all three).
__global__ void merge_shards_kernel(const int32_t *__restrict__ ids, const float *__restrict__ scores,
                                    const int32_t *__restrict__ tokens, size_t stride_ids, size_t stride_scores,
                                    size_t stride_tokens, const long long *__restrict__ offsets,
                                    int P, int B, int n, int L, int32_t *__restrict__ out_ids,
                                    float *__restrict__ out_scores, int32_t *__restrict__ out_tokens)
{
    const int b = blockIdx.x, lane = threadIdx.x;
    unsigned long long m = 0ull;
    for (int p = 0; p < P; ++p) {
        unsigned long long v = 0ull;
        if (lane < n) {
            const int32_t id = ids[p * stride_ids + (size_t)b * n + lane];
            if (id >= 0) v = pack_candidate(scores[p * stride_scores + (size_t)b * n + lane], (uint32_t)(id + offsets[p]));
        }
        // a shard's list is sorted with its missing entries (id -1) last, so it is a valid input
        m = warp_merge_top32(m, v, lane);
    }
    if (lane >= n) m = 0ull;
    const long long gid = m ? (long long)candidate_id(m) : -1;
    if (lane < n) {
        out_ids[(size_t)b * n + lane] = (int32_t)gid;
        out_scores[(size_t)b * n + lane] = m ? candidate_score(m) : -INFINITY;
    }
    // where did this winner come from?  shard = last offset <= gid; slot = its rank there
    int p = -1, r = -1;
    if (gid >= 0) {
        p = 0;
        while (p + 1 < P && offsets[p + 1] <= gid) ++p;
        const int32_t local = (int32_t)(gid - offsets[p]);
        for (int k = 0; k < n; ++k)
            if (ids[p * stride_ids + (size_t)b * n + k] == local) { r = k; break; }
    }
    if (lane < n)
        for (int t = 0; t < L; ++t)
            out_tokens[((size_t)b * n + lane) * L + t] =
                r >= 0 ? tokens[p * stride_tokens + (((size_t)b * n + r) * L + t)] : -1;
}

}  // namespace

cudaError_t launch_merge_shards(const int32_t *ids, const float *scores, const int32_t *tokens, size_t stride_ids,
                                size_t stride_scores, size_t stride_tokens, const long long *offsets, int P, int B,
                                int n, int L, int32_t *out_ids, float *out_scores, int32_t *out_tokens,
                                cudaStream_t stream)
{
    merge_shards_kernel<<<B, 32, 0, stream>>>(ids, scores, tokens, stride_ids, stride_scores, stride_tokens, offsets, P, B,
                                              n, L, out_ids, out_scores, out_tokens);
    return cudaGetLastError();
}

}  // namespace dresd

// K4 -- grid-level merge: the per-CTA sorted candidate lists of one query are
// folded into the final top-n (Eq. 3's arg max over the whole datastore,
// extended to the n best; ties to the lower row index).
// K5 -- value lookup f_D of Section 3.5: copy the first draft_len stored
// continuation tokens of every selected key into the n x L draft matrix.
// Both run in one kernel: the CTA that merged a query's lists gathers its tokens.
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kMergeWarps = 16;

// One CTA per query.  Each warp folds every 16th per-CTA list (eight loads in flight before
// the dependent merge chain), the 16 partial lists are folded pairwise in four rounds, and --
// fused K5 -- the whole CTA then copies the winners' stored tokens.  Probe pass (gtau set):
// only the n-th best score is kept, as the grid-wide filter word.
__global__ void __launch_bounds__(kMergeWarps * 32)
merge_gather_kernel(const unsigned long long *__restrict__ cand, int lists, int B, int top_n,
                    int32_t *__restrict__ out_ids, float *__restrict__ out_scores, unsigned int *__restrict__ gtau,
                    const int32_t *__restrict__ next_tokens, int stored_len, long long N, int draft_len,
                    int32_t *__restrict__ out_tokens, int *status)
{
    __shared__ unsigned long long part[kMergeWarps][kListLen];
    __shared__ int win[kListLen];
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_wait();                           // the scan's lists are complete and visible
    pdl_launch_dependents();

    unsigned long long m = 0ull;
    // eight lists in flight per warp before the dependent merge chain; empty lists (CTAs that saw
    // no candidate: short scans, token windows) are skipped
    for (int g0 = warp; g0 < lists; g0 += 8 * kMergeWarps) {
        unsigned long long l[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int g = g0 + k * kMergeWarps;
            l[k] = g < lists ? cand[((size_t)g * B + b) * kCandStride + lane] : 0ull;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (shfl_u64(l[k], 0) != 0ull) m = warp_merge_top32(m, l[k], lane);      // sorted: slot 0 is the best
    }
    part[warp][lane] = m;
    __syncthreads();
    for (int span = kMergeWarps / 2; span >= 1; span >>= 1) {
        if (warp < span) {
            m = warp_merge_top32(part[warp][lane], part[warp + span][lane], lane);
            part[warp][lane] = m;
        }
        __syncthreads();
    }
    m = part[0][lane];
    if (gtau) {                           // probe pass: publish the n-th best as the filter
        if (warp == 0 && lane == top_n - 1) gtau[b] = m ? float_to_ordered(candidate_score(m)) : 0u;
        return;
    }
    if (warp == 0 && lane < top_n) {
        int id = m ? (int32_t)candidate_id(m) : -1;
        if (!debug_check(id >= -1 && id < N, status, 41)) id = -1;     // debug build: a winner is a row of the store
        out_ids[(size_t)b * top_n + lane] = id;
        out_scores[(size_t)b * top_n + lane] = m ? candidate_score(m) : -INFINITY;
        win[lane] = id;
    }
    __syncthreads();
    // K5: the first draft_len stored tokens of every winner (Section 3.5, f_D: k -> v)
    const int total = top_n * draft_len;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int r = i / draft_len, t = i - r * draft_len;
        const long long id = win[r];
        out_tokens[(size_t)b * total + i] = (id >= 0 && id < N) ? next_tokens[(size_t)id * stored_len + t] : -1;
    }
}

// Compact copy of the first stored token of every key (the column the first-token
// filter of Section 3.5 tests), so that the scan reads 4 bytes per row for it.
__global__ void extract_first_kernel(const int32_t *__restrict__ next_tokens, int stored_len, long long N,
                                     int32_t *__restrict__ first_col)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < N;
         i += (long long)gridDim.x * blockDim.x)
        first_col[i] = next_tokens[i * stored_len];
}

// Index of a store sorted by first token (Section 3.5: only keys whose value starts with
// x_{t+1} can be drafted, so a sorted store needs to be scanned over that token's rows only).
__global__ void check_sorted_kernel(const int32_t *__restrict__ first_col, long long N, int *flag)
{
    int bad = 0;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < N;
         i += (long long)gridDim.x * blockDim.x) {
        const int cur = first_col[i];
        if (cur < 0) bad |= 2;
        if (i > 0 && first_col[i - 1] > cur) bad |= 1;
    }
    if (bad) atomicOr(flag, bad);
}

// Row i opens the windows of every token in (first_col[i-1], first_col[i]]: tokens without
// rows get an empty window at the next present token's first row.  Sorted input only.
__global__ void build_windows_kernel(const int32_t *__restrict__ first_col, long long N, int vocab,
                                     int32_t *__restrict__ win_start)
{
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i <= N;
         i += (long long)gridDim.x * blockDim.x) {
        if (i == N) {
            win_start[vocab] = (int32_t)N;
            continue;
        }
        const int prev = i > 0 ? first_col[i - 1] : -1, cur = first_col[i];
        for (int t = prev + 1; t <= cur && t < vocab; ++t) win_start[t] = (int32_t)i;
    }
}

}  // namespace

cudaError_t launch_check_sorted(const int32_t *first_col, long long N, int *flag, cudaStream_t stream)
{
    long long blocks = (N + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    check_sorted_kernel<<<(int)blocks, 256, 0, stream>>>(first_col, N, flag);
    return cudaGetLastError();
}

cudaError_t launch_build_windows(const int32_t *first_col, long long N, int vocab, int32_t *win_start,
                                 cudaStream_t stream)
{
    long long blocks = (N + 1 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    build_windows_kernel<<<(int)blocks, 256, 0, stream>>>(first_col, N, vocab, win_start);
    return cudaGetLastError();
}

cudaError_t launch_extract_first(const int32_t *next_tokens, int stored_len, long long N, int32_t *first_col,
                                 cudaStream_t stream)
{
    const int threads = 256;
    long long blocks = (N + threads - 1) / threads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    extract_first_kernel<<<(int)blocks, threads, 0, stream>>>(next_tokens, stored_len, N, first_col);
    return cudaGetLastError();
}

__global__ void debug_selftest_kernel(int *status)
{
    const int index = 5, limit = 4;                    // an index that is out of range; the access is skipped
    if (debug_check(index < limit, status, 7)) status[index] = 0;
}

cudaError_t launch_debug_selftest(int *status, cudaStream_t stream)
{
    debug_selftest_kernel<<<1, 1, 0, stream>>>(status);
    return cudaGetLastError();
}

cudaError_t launch_merge_gather(const unsigned long long *cand, int lists, int B, int top_n, int32_t *out_ids,
                                float *out_scores, const int32_t *next_tokens, int stored_len, long long N,
                                int draft_len, int32_t *out_tokens, cudaStream_t stream, int *status)
{
    return launch_dependent(merge_gather_kernel, dim3(B), dim3(kMergeWarps * 32), 0, stream, cand, lists, B, top_n, out_ids,
                            out_scores, (unsigned int *)nullptr, next_tokens, stored_len, N, draft_len, out_tokens, status);
}

cudaError_t launch_merge_tau(const unsigned long long *cand, int lists, int B, int top_n, unsigned int *gtau,
                             cudaStream_t stream)
{
    return launch_dependent(merge_gather_kernel, dim3(B), dim3(kMergeWarps * 32), 0, stream, cand, lists, B, top_n,
                            (int32_t *)nullptr, (float *)nullptr, gtau, (const int32_t *)nullptr, 0, 0LL, 0,
                            (int32_t *)nullptr, (int *)nullptr);
}

}  // namespace dresd

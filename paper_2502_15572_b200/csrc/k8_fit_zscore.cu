// K8 -- the statistics of Eq. 1 (Section 3.2 of the paper): E[V] and Var[V] per embedding
// dimension, estimated from a sample V of N full-size token embeddings (the paper samples
// about a million).  One streaming pass over N x d_in 16-bit values: HBM-bound.
//
// Arithmetic.  A per-column shift K_j (a trimmed fp32 mean of the first <= 32 rows, computed once by
// a small kernel so that every CTA uses the same bits) is subtracted before anything is summed:
//     S1_j = sum_i (x_ij - K_j),   S2_j = sum_i (x_ij - K_j)^2,
//     E_j = K_j + S1_j / N,        Var_j = S2_j / N - (S1_j / N)^2      (population variance),
// so the subtraction in Var_j cancels almost nothing even when |E_j| >> sigma_j.  A thread sums
// at most 64 rows in fp32, then folds the chunk into float64; partial sums of the row slices are
// written out and added in a fixed order by the last kernel (the result is run-to-run identical).
//
// Layout: a thread owns 8 adjacent columns (one 16-byte load per row); the threads of a CTA
// cover up to 2048 adjacent columns, narrower samples put several row lanes side by side.
// Eight rows are in flight per thread, two CTAs per SM.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "internal.h"

namespace dresd {
namespace {

constexpr int kFitThreads = 256;
constexpr int kFitChunk = 64;      // rows a thread sums in fp32 before folding into float64
constexpr int kFitUnroll = 8;      // rows in flight per thread
constexpr int kShiftRows = 32;

template <typename T> __device__ __forceinline__ void unpack8(const uint4 &v, float *x);
template <> __device__ __forceinline__ void unpack8<__half>(const uint4 &v, float *x)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
}
template <> __device__ __forceinline__ void unpack8<__nv_bfloat16>(const uint4 &v, float *x)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// shift[j] = fp32 mean of column j over the first min(N, 32) rows, without the largest and the
// smallest of them when there are at least three (one outlier row must not drag the shift away).
template <typename T>
__global__ void fit_shift_kernel(const T *__restrict__ V, long long N, int d_in, float *__restrict__ shift)
{
    const int g = blockIdx.x * blockDim.x + threadIdx.x;      // column group
    if (g * 8 >= d_in) return;
    const int rows = (int)(N < kShiftRows ? N : kShiftRows);
    float s[8], lo[8], hi[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        s[i] = 0.f;
        lo[i] = INFINITY;
        hi[i] = -INFINITY;
    }
    for (int r = 0; r < rows; ++r) {
        const uint4 v = *reinterpret_cast<const uint4 *>(V + (size_t)r * d_in + (size_t)g * 8);
        float x[8];
        unpack8<T>(v, x);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            s[i] += x[i];
            lo[i] = fminf(lo[i], x[i]);
            hi[i] = fmaxf(hi[i], x[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float k = rows >= 3 ? (s[i] - lo[i] - hi[i]) / (float)(rows - 2) : s[i] / (float)rows;
        if (!(fabsf(k) <= 3.0e38f)) k = 0.f;                  // non-finite input: any shift is as good
        shift[g * 8 + i] = k;
    }
}

struct FitArgs {
    long long N;
    int d_in;
    int groups;          // column groups of 8 = d_in / 8
    int cb;              // column groups per CTA (<= 256)
    int lanes;           // row lanes per CTA = 256 / cb
    int slices;          // gridDim.y
    const float *shift;  // [d_in]
    double *part;        // [slices][d_in][2]
};

template <typename T>
__global__ void __launch_bounds__(kFitThreads, 2) fit_sums_kernel(const T *__restrict__ V, const FitArgs a)
{
    __shared__ double red[kFitThreads * 16];
    const int tid = threadIdx.x;
    const int lane_r = tid / a.cb;                      // row lane of this thread
    const int g = blockIdx.x * a.cb + tid % a.cb;       // its column group
    const bool active = lane_r < a.lanes && g < a.groups;
    const long long per = (a.N + a.slices - 1) / a.slices;
    const long long begin = (long long)blockIdx.y * per;
    const long long end = begin + per < a.N ? begin + per : a.N;

    double acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.0;
    if (active) {
        float K[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) K[i] = a.shift[g * 8 + i];
        const size_t stride = (size_t)a.lanes * a.d_in;                       // elements between my rows
        long long row = begin + lane_r;
        const T *p = V + (size_t)row * a.d_in + (size_t)g * 8;
        while (row < end) {
            float s[8], q[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) s[i] = q[i] = 0.f;
            for (int u = 0; u < kFitChunk && row < end; u += kFitUnroll) {
                uint4 v[kFitUnroll];
                bool ok[kFitUnroll];
#pragma unroll
                for (int k = 0; k < kFitUnroll; ++k) {
                    ok[k] = row + (long long)k * a.lanes < end;
                    v[k] = ok[k] ? __ldcs(reinterpret_cast<const uint4 *>(p + (size_t)k * stride)) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int k = 0; k < kFitUnroll; ++k) {
                    if (ok[k]) {
                        float x[8];
                        unpack8<T>(v[k], x);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float t = x[i] - K[i];
                            s[i] += t;
                            q[i] = fmaf(t, t, q[i]);
                        }
                    }
                }
                row += (long long)kFitUnroll * a.lanes;
                p += (size_t)kFitUnroll * stride;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                acc[i] += (double)s[i];
                acc[8 + i] += (double)q[i];
            }
        }
    }
    // fold the row lanes (fixed order), then one partial per slice and column
    if (a.lanes > 1) {
#pragma unroll
        for (int i = 0; i < 16; ++i) red[tid * 16 + i] = acc[i];
        __syncthreads();
        if (active && lane_r == 0) {
            for (int l = 1; l < a.lanes; ++l)
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] += red[(l * a.cb + tid) * 16 + i];
        }
    }
    if (active && lane_r == 0) {
        double *out = a.part + ((size_t)blockIdx.y * a.d_in + (size_t)g * 8) * 2;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            out[2 * i] = acc[i];
            out[2 * i + 1] = acc[8 + i];
        }
    }
}

__global__ void fit_final_kernel(const double *__restrict__ part, const float *__restrict__ shift, int slices,
                                 int d_in, long long N, float *__restrict__ mean, float *__restrict__ var)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d_in) return;
    double s1 = 0.0, s2 = 0.0;
    for (int s = 0; s < slices; ++s) {
        s1 += part[((size_t)s * d_in + j) * 2];
        s2 += part[((size_t)s * d_in + j) * 2 + 1];
    }
    const double m = s1 / (double)N;
    double v = s2 / (double)N - m * m;
    if (v < 0.0) v = 0.0;
    mean[j] = (float)((double)shift[j] + m);
    var[j] = (float)v;
}

void fit_plan(long long N, int d_in, int sms, FitArgs *a, int *col_blocks)
{
    a->N = N;
    a->d_in = d_in;
    a->groups = d_in / 8;
    a->cb = a->groups < kFitThreads ? a->groups : kFitThreads;
    a->lanes = kFitThreads / a->cb;
    *col_blocks = (a->groups + a->cb - 1) / a->cb;
    long long slices = (2LL * sms + *col_blocks - 1) / *col_blocks;
    const long long max_slices = (N + a->lanes - 1) / a->lanes;          // at least one row per lane group
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    a->slices = (int)slices;
}

}  // namespace

size_t fit_zscore_workspace_bytes(long long N, int d_in, int sms)
{
    FitArgs a{};
    int cbk = 0;
    fit_plan(N, d_in, sms, &a, &cbk);
    return 256 + (((size_t)d_in * sizeof(float) + 255) & ~(size_t)255) + (size_t)a.slices * d_in * 2 * sizeof(double);
}

cudaError_t launch_fit_zscore(const void *V, int dtype, long long N, int d_in, int sms, void *workspace,
                              float *mean, float *var, cudaStream_t stream)
{
    FitArgs a{};
    int col_blocks = 0;
    fit_plan(N, d_in, sms, &a, &col_blocks);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    float *shift = reinterpret_cast<float *>(ws);
    double *part = reinterpret_cast<double *>(ws + (((size_t)d_in * sizeof(float) + 255) & ~(size_t)255));
    a.shift = shift;
    a.part = part;
    const dim3 grid(col_blocks, a.slices);
    const int sgrid = (a.groups + 127) / 128;
    if (dtype == kF16) {
        fit_shift_kernel<__half><<<sgrid, 128, 0, stream>>>(static_cast<const __half *>(V), N, d_in, shift);
        fit_sums_kernel<__half><<<grid, kFitThreads, 0, stream>>>(static_cast<const __half *>(V), a);
    } else {
        fit_shift_kernel<__nv_bfloat16><<<sgrid, 128, 0, stream>>>(static_cast<const __nv_bfloat16 *>(V), N, d_in, shift);
        fit_sums_kernel<__nv_bfloat16><<<grid, kFitThreads, 0, stream>>>(static_cast<const __nv_bfloat16 *>(V), a);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    fit_final_kernel<<<(d_in + 255) / 256, 256, 0, stream>>>(part, shift, a.slices, d_in, N, mean, var);
    return cudaGetLastError();
}

}  // namespace dresd

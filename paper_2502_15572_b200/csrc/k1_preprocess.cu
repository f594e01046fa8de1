// K1 -- query preprocessing, Algorithm 1 steps 4-6 of the paper:
//   Eq. 1   v <- (v - E[V]) / sqrt(Var[V] + eps)        (optional)
//   Sec 3.3 v_l <- v W_l (after an optional centring)     (optional)
//   Eq. 2   v_l <- v_l / max(||v_l||_2, eps)
// One CTA per query.  Besides the fp32 unit query it emits, for 16-bit
// datastores, the two-term split q = hi + lo/scale in the store dtype that the
// tensor-core scoring kernels use as their B operand (row 2b = hi, 2b+1 = lo,
// zero-padded to a multiple of 64 columns), so that scoring with 16-bit
// operands keeps fp32-level accuracy.
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__half>(__half x) { return __half2float(x); }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x)
{
    return __bfloat162float(x);
}
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ __half from_f32<__half>(float x) { return __float2half_rn(x); }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x)
{
    return __float2bfloat16_rn(x);
}
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }

constexpr int kThreads = 1024;

__device__ __forceinline__ float block_sum(float x, float *scratch /*[32]*/)
{
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    __syncthreads();                      // scratch may still be read from a previous call
    if (lane == 0) scratch[warp] = x;
    __syncthreads();
    float t = (lane < (blockDim.x >> 5)) ? scratch[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    return t;                             // every thread holds the total
}

template <typename T>
__global__ void __launch_bounds__(kThreads) preprocess_kernel(PreprocessArgs a)
{
    extern __shared__ float smem_f[];
    float *v = smem_f;                    // [d_in]
    float *vl = v + a.d_in;               // [d]
    float *part = vl + a.d;               // [slices][d] (projection only)
    __shared__ float red[32];

    const int b = blockIdx.x;
    const int tid = threadIdx.x;
    // operand rows of query b: (2b, 2b+1), or -- blocked layout -- rows (b % 8) and 8 + (b % 8)
    // of the 16-row block b / 8, so that a 16-lane TMEM fragment holds hi and lo of 8 queries
    const int row_hi = a.split_blocked ? 16 * (b >> 3) + (b & 7) : 2 * b;
    const int row_lo = a.split_blocked ? row_hi + 8 : row_hi + 1;
    T *split_hi = a.qsplit ? static_cast<T *>(a.qsplit) + (size_t)row_hi * a.dpad : nullptr;
    T *split_lo = a.qsplit ? static_cast<T *>(a.qsplit) + (size_t)row_lo * a.dpad : nullptr;
    float *qrow = a.qhat + (size_t)b * a.d;
    if (tid == 0 && a.gtau) a.gtau[b] = 0u;          // fresh grid-wide filter for this call

    if (b >= a.B) {                       // padding rows of the operand: zeros
        for (int c = tid; c < a.d; c += blockDim.x) qrow[c] = 0.f;
        if (split_hi)
            for (int c = tid; c < a.dpad; c += blockDim.x) {
                split_hi[c] = from_f32<T>(0.f);
                split_lo[c] = from_f32<T>(0.f);
            }
        return;
    }

    const T *q = static_cast<const T *>(a.queries) + (size_t)b * a.d_in;
    for (int j = tid; j < a.d_in; j += blockDim.x) {
        float x = to_f32<T>(q[j]);
        if (a.mean) x = (x - a.mean[j]) / sqrtf(a.var[j] + a.eps_z);      // Eq. 1
        if (a.W && a.pca_mean) x -= a.pca_mean[j];
        v[j] = x;
    }
    __syncthreads();

    if (a.W) {                                                             // v_l = v W
        // Threads are arranged [slice][column]: consecutive threads read
        // consecutive columns of one W row (coalesced); slices split d_in.
        int ct = 1;
        while (ct * 2 <= a.d && ct * 2 <= (int)blockDim.x) ct *= 2;
        const int slices = blockDim.x / ct;
        const int slice = tid / ct, cl = tid % ct;
        const int jper = (a.d_in + slices - 1) / slices;
        const int j0 = slice * jper, j1 = min(a.d_in, j0 + jper);
        const T *W = static_cast<const T *>(a.W);
        for (int c = cl; c < a.d; c += ct) {
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
            int j = j0;
            for (; j + 3 < j1; j += 4) {
                acc0 = fmaf(v[j + 0], to_f32<T>(W[(size_t)(j + 0) * a.d + c]), acc0);
                acc1 = fmaf(v[j + 1], to_f32<T>(W[(size_t)(j + 1) * a.d + c]), acc1);
                acc2 = fmaf(v[j + 2], to_f32<T>(W[(size_t)(j + 2) * a.d + c]), acc2);
                acc3 = fmaf(v[j + 3], to_f32<T>(W[(size_t)(j + 3) * a.d + c]), acc3);
            }
            for (; j < j1; ++j) acc0 = fmaf(v[j], to_f32<T>(W[(size_t)j * a.d + c]), acc0);
            part[(size_t)slice * a.d + c] = (acc0 + acc1) + (acc2 + acc3);
        }
        __syncthreads();
        for (int c = tid; c < a.d; c += blockDim.x) {
            float s = 0.f;
            for (int sl = 0; sl < slices; ++sl) s += part[(size_t)sl * a.d + c];
            vl[c] = s;
        }
    } else {
        for (int c = tid; c < a.d; c += blockDim.x) vl[c] = v[c];
    }
    __syncthreads();

    float ss = 0.f;                                                        // Eq. 2
    for (int c = tid; c < a.d; c += blockDim.x) ss = fmaf(vl[c], vl[c], ss);
    ss = block_sum(ss, red);
    const float den = fmaxf(sqrtf(ss), a.eps_n);

    for (int c = tid; c < a.dpad; c += blockDim.x) {
        float x = c < a.d ? vl[c] / den : 0.f;
        if (c < a.d) qrow[c] = x;
        if (split_hi) {
            T hi = from_f32<T>(x);
            float r = (x - to_f32<T>(hi)) * a.lo_scale;
            split_hi[c] = hi;
            split_lo[c] = from_f32<T>(r);
        }
    }
}

}  // namespace

cudaError_t launch_preprocess(const PreprocessArgs &a, cudaStream_t stream)
{
    if (a.rows <= 0) return cudaSuccess;
    int ct = 1;
    while (ct * 2 <= a.d && ct * 2 <= kThreads) ct *= 2;
    const int slices = a.W ? kThreads / ct : 0;
    size_t smem = sizeof(float) * ((size_t)a.d_in + a.d + (size_t)slices * a.d);
    cudaError_t e = cudaSuccess;
    auto go = [&](auto kernel) {
        if (smem > 48 * 1024)
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return;
        kernel<<<a.rows, kThreads, smem, stream>>>(a);
        e = cudaGetLastError();
    };
    switch (a.dtype) {
    case kF32: go(preprocess_kernel<float>); break;
    case kF16: go(preprocess_kernel<__half>); break;
    default: go(preprocess_kernel<__nv_bfloat16>); break;
    }
    return e;
}

}  // namespace dresd

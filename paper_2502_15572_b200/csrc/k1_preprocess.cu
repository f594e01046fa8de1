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

// K1a -- the projection v W of ALL queries of the call, split over d_in: CTA s takes the
// rows [s * rps, (s+1) * rps) of W (read once, coalesced, for every query), applies Eq. 1 and
// the centring to the matching slice of each query, and writes the partial products
// partial[s][b][c].  K1b adds the slices in a fixed order, so the result does not depend on
// the launch.  (One CTA per query reading all of W, as K1b does without a workspace, is
// latency-bound: 130 us for 16 queries x 4096 x 256; this form takes a few microseconds.)
constexpr int kProjThreads = 256;
constexpr int kProjWarps = kProjThreads / 32;

template <typename T> struct ProjVec;    // 16 bytes of a W row
template <> struct ProjVec<float> { static constexpr int N = 4; };
template <> struct ProjVec<__half> { static constexpr int N = 8; };
template <> struct ProjVec<__nv_bfloat16> { static constexpr int N = 8; };
template <typename T> __device__ __forceinline__ void unpack_w(const uint4 &v, float *w);
template <> __device__ __forceinline__ void unpack_w<float>(const uint4 &v, float *w)
{
    w[0] = __uint_as_float(v.x); w[1] = __uint_as_float(v.y); w[2] = __uint_as_float(v.z); w[3] = __uint_as_float(v.w);
}
template <> __device__ __forceinline__ void unpack_w<__half>(const uint4 &v, float *w)
{
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&u[i]));
        w[2 * i] = f.x;
        w[2 * i + 1] = f.y;
    }
}
template <> __device__ __forceinline__ void unpack_w<__nv_bfloat16>(const uint4 &v, float *w)
{
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        w[2 * i] = __uint_as_float(u[i] << 16);
        w[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
    }
}

// The CTA first copies its slice of W to shared memory with every 16-byte load in flight at
// once (W does not survive in L2 between calls -- the scan streams gigabytes through it -- so
// these are DRAM reads, and a loop that waits for each row costs ~1.2 k cycles per row).  Then
// warp w takes the queries w, w + 8, ... (at most 8 of the 64) and a lane 16 bytes (4 or 8
// columns) of every row; no sum crosses a warp.
// QW = queries per warp (1, 2, 4 or 8, chosen from B): the inner loops are branch-free.
template <typename T, int QW>
__global__ void __launch_bounds__(kProjThreads) project_partial_kernel(PreprocessArgs a)
{
    constexpr int VEC = ProjVec<T>::N;
    extern __shared__ __align__(16) uint8_t proj_smem[];
    const int rps = a.rows_per_slice;
    const int s = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int j0 = s * rps, nr = min(a.d_in, j0 + rps) - j0;
    uint4 *ws = reinterpret_cast<uint4 *>(proj_smem);                        // [nr][d / VEC]: the slice of W
    float *vs = reinterpret_cast<float *>(proj_smem + (size_t)rps * a.d * sizeof(T));   // [B][rps]: the queries' slices
    const int cblocks = a.d / VEC;        // 16-byte column blocks per row (d is a multiple of VEC)
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const T *>(a.W) + (size_t)j0 * a.d);
        const int total = nr * cblocks;
        for (int i0 = tid; i0 < total; i0 += 8 * kProjThreads) {
            uint4 v[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const int i = i0 + r * kProjThreads;
                v[r] = i < total ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                const int i = i0 + r * kProjThreads;
                if (i < total) ws[i] = v[r];
            }
        }
    }
    const T *Q = static_cast<const T *>(a.queries);
    for (int i = tid; i < a.B * rps; i += kProjThreads) {
        const int b = i / rps, jj = i - b * rps;
        float x = 0.f;
        if (jj < nr) {
            const int j = j0 + jj;
            x = to_f32<T>(Q[(size_t)b * a.d_in + j]);
            if (a.mean) x = (x - a.mean[j]) / sqrtf(a.var[j] + a.eps_z);      // Eq. 1
            if (a.pca_mean) x -= a.pca_mean[j];
        }
        vs[i] = x;
    }
    __syncthreads();
    if (warp >= a.B) return;
    int qrow[QW];                         // my queries w, w + 8, ...; past B: the last one again (not stored)
#pragma unroll
    for (int u = 0; u < QW; ++u) qrow[u] = min(warp + kProjWarps * u, a.B - 1) * rps;
    for (int cb = lane; cb < cblocks; cb += 32) {
        float acc[QW][VEC];
#pragma unroll
        for (int u = 0; u < QW; ++u)
#pragma unroll
            for (int k = 0; k < VEC; ++k) acc[u][k] = 0.f;
#pragma unroll 4
        for (int jj = 0; jj < nr; ++jj) {
            float w[VEC];
            unpack_w<T>(ws[jj * cblocks + cb], w);
#pragma unroll
            for (int u = 0; u < QW; ++u) {
                const float x = vs[qrow[u] + jj];
#pragma unroll
                for (int k = 0; k < VEC; ++k) acc[u][k] = fmaf(x, w[k], acc[u][k]);
            }
        }
#pragma unroll
        for (int u = 0; u < QW; ++u) {
            const int b = warp + kProjWarps * u;
            if (b < a.B) {
                float *o = a.partial + ((size_t)s * a.B + b) * a.d + (size_t)cb * VEC;
#pragma unroll
                for (int k = 0; k < VEC; k += 4)
                    *reinterpret_cast<float4 *>(o + k) = make_float4(acc[u][k], acc[u][k + 1], acc[u][k + 2], acc[u][k + 3]);
            }
        }
    }
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
    pdl_launch_dependents();              // the scan may set itself up while this kernel runs
    // operand rows of query b: (2b, 2b+1), or -- blocked layout -- rows (b % 8) and 8 + (b % 8)
    // of the 16-row block b / 8, so that a 16-lane TMEM fragment holds hi and lo of 8 queries
    // or -- merged layout -- rows b and rows + b, both terms scaled by lo_scale;
    // or -- packed layout, two 32-element keys per 64-element store row -- rows 4b .. 4b+3 =
    // (hi|0), (lo|0), (0|hi), (0|lo): two column pairs that score the even and the odd key of a row
    // or -- halves layout -- rows b (hi) and rows + b (lo), the hi rows of all queries first
    const bool merged = a.split_blocked == 2, packed = a.split_blocked == 3, halves = a.split_blocked == 4;
    const int row_hi = packed ? 4 * b : (merged || halves) ? b : a.split_blocked ? 16 * (b >> 3) + (b & 7) : 2 * b;
    const int row_lo = (merged || halves) ? a.rows + b : a.split_blocked == 1 ? row_hi + 8 : row_hi + 1;
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
                if (packed) {
                    split_hi[2 * a.dpad + c] = from_f32<T>(0.f);
                    split_lo[2 * a.dpad + c] = from_f32<T>(0.f);
                }
            }
        if (a.qsplit8)
            for (int c = tid; c < a.dpad8; c += blockDim.x) store_query_e4m3(a.qsplit8, a.dpad8, a.pack2, b, c, 0.f);
        return;
    }

    const T *q = static_cast<const T *>(a.queries) + (size_t)b * a.d_in;
    const bool presummed = a.W && a.partial;             // K1a has done Eq. 1 and the products
    for (int j = tid; j < a.d_in && !presummed; j += blockDim.x) {
        float x = to_f32<T>(q[j]);
        if (a.mean) x = (x - a.mean[j]) / sqrtf(a.var[j] + a.eps_z);      // Eq. 1
        if (a.W && a.pca_mean) x -= a.pca_mean[j];
        v[j] = x;
    }
    __syncthreads();

    if (presummed) {                                                       // v_l = sum of K1a's slices
        // threads arranged [group][column]: group g adds slices g, g + groups, ... (loads of
        // different slices in flight together), then the groups' sums are added in order
        int ct = 1;
        while (ct * 2 <= a.d && ct * 2 <= (int)blockDim.x) ct *= 2;
        const int groups = blockDim.x / ct;
        const int grp = tid / ct, cl = tid % ct;
        for (int c = cl; c < a.d; c += ct) {
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
            int sl = grp;
            for (; sl + 3 * groups < a.slices; sl += 4 * groups) {
                s0 += a.partial[((size_t)(sl + 0 * groups) * a.B + b) * a.d + c];
                s1 += a.partial[((size_t)(sl + 1 * groups) * a.B + b) * a.d + c];
                s2 += a.partial[((size_t)(sl + 2 * groups) * a.B + b) * a.d + c];
                s3 += a.partial[((size_t)(sl + 3 * groups) * a.B + b) * a.d + c];
            }
            for (; sl < a.slices; sl += groups) s0 += a.partial[((size_t)sl * a.B + b) * a.d + c];
            part[(size_t)grp * a.d + c] = (s0 + s1) + (s2 + s3);
        }
        __syncthreads();
        for (int c = tid; c < a.d; c += blockDim.x) {
            float t = 0.f;
            for (int g = 0; g < groups; ++g) t += part[(size_t)g * a.d + c];
            vl[c] = t;
        }
    } else if (a.W) {                                                      // v_l = v W
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
            if (merged) hi = from_f32<T>(to_f32<T>(hi) * a.lo_scale);     // exact: a power of two, |hi| <= 1
            if (packed) {
                // c < 32: the query's element c, for the even key (columns c) and the odd key (columns 32 + c);
                // the other half of every operand row is zero
                if (c < 32) {
                    const T z = from_f32<T>(0.f), lo = from_f32<T>(r);
                    split_hi[c] = hi;
                    split_hi[32 + c] = z;
                    split_lo[c] = lo;
                    split_lo[32 + c] = z;
                    split_hi[2 * a.dpad + c] = z;
                    split_hi[2 * a.dpad + 32 + c] = hi;
                    split_lo[2 * a.dpad + c] = z;
                    split_lo[2 * a.dpad + 32 + c] = lo;
                }
                continue;
            }
            split_hi[c] = hi;
            split_lo[c] = from_f32<T>(r);
        }
    }
    if (a.qsplit8)                                       // the two 8-bit terms of the quantised search
        for (int c = tid; c < a.dpad8; c += blockDim.x)
            store_query_e4m3(a.qsplit8, a.dpad8, a.pack2, b, c, c < a.d ? vl[c] / den : 0.f);
}

}  // namespace

void preprocess_split_plan(int d_in, int d, int B, int elem_bytes, size_t bytes, int *slices, int *rows_per_slice)
{
    *slices = 0;
    *rows_per_slice = 0;
    if (B <= 0 || bytes == 0) return;
    const size_t per_slice = sizeof(float) * (size_t)B * d;
    const long long cap = (long long)(bytes / per_slice);
    if (cap < 2) return;                                  // no room: the unsplit form runs
    // a CTA holds its slice of W (rows x d) and of the queries (B x rows) in 48 KB of shared memory
    auto fits = [&](int rps) { return (size_t)rps * d * elem_bytes + sizeof(float) * (size_t)B * rps <= 48 * 1024; };
    int rps = 64;
    while (rps > 1 && !fits(rps)) rps /= 2;
    if (!fits(rps)) return;
    const long long n = (d_in + rps - 1) / rps;
    if (n > cap || n > 1024) return;                      // too many slices for the workspace: unsplit form
    *slices = (int)n;
    *rows_per_slice = rps;
}

cudaError_t launch_preprocess(const PreprocessArgs &a, cudaStream_t stream)
{
    if (a.rows <= 0) return cudaSuccess;
    if (a.W && a.partial && a.B > 0) {
        const size_t eb = a.dtype == kF32 ? 4 : 2;
        const size_t psm = (size_t)a.rows_per_slice * a.d * eb + sizeof(float) * (size_t)a.B * a.rows_per_slice;
        const int per_warp = (a.B + kProjWarps - 1) / kProjWarps;
        const int qw = per_warp <= 1 ? 1 : per_warp <= 2 ? 2 : per_warp <= 4 ? 4 : 8;
        auto launch = [&](auto k1, auto k2, auto k4, auto k8) {
            if (qw == 1) k1<<<a.slices, kProjThreads, psm, stream>>>(a);
            else if (qw == 2) k2<<<a.slices, kProjThreads, psm, stream>>>(a);
            else if (qw == 4) k4<<<a.slices, kProjThreads, psm, stream>>>(a);
            else k8<<<a.slices, kProjThreads, psm, stream>>>(a);
        };
        switch (a.dtype) {
        case kF32:
            launch(project_partial_kernel<float, 1>, project_partial_kernel<float, 2>,
                   project_partial_kernel<float, 4>, project_partial_kernel<float, 8>);
            break;
        case kF16:
            launch(project_partial_kernel<__half, 1>, project_partial_kernel<__half, 2>,
                   project_partial_kernel<__half, 4>, project_partial_kernel<__half, 8>);
            break;
        default:
            launch(project_partial_kernel<__nv_bfloat16, 1>, project_partial_kernel<__nv_bfloat16, 2>,
                   project_partial_kernel<__nv_bfloat16, 4>, project_partial_kernel<__nv_bfloat16, 8>);
            break;
        }
        cudaError_t pe = cudaGetLastError();
        if (pe != cudaSuccess) return pe;
    }
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

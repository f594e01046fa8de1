// dresd_retrieve_noalloc -- the retrieval call for callers that must not
// allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need a
// draft: a serving runtime that hands all device memory to its own pool at
// start-up and forbids further driver allocations, a plug-in that runs inside
// somebody else's memory budget, or code on a latency-critical path where an
// allocation's implicit device synchronisation is not acceptable.  The regular
// path needs a workspace (the unit queries, their 16-bit split, and the
// per-CTA candidate lists that the scoring kernel hands to the merge kernel)
// and gets it from cudaMalloc in dresd_store_create().  This entry point keeps
// that workspace in a fixed array that is part of the library image instead:
// every GPU that loads the library holds kScratchBytes (about 576 KB) of it
// until the process exits, and nothing is ever allocated or freed.
//
// The price is a smaller envelope (B <= 8 queries per call) and one shared
// workspace: calls that overlap on the GPU race on it.
#include <mutex>

#include "../../include/dresd.h"
#include "internal.h"

using namespace dresd;

namespace {

constexpr int kNaMaxBatch = DRESD_NOALLOC_MAX_BATCH;   // queries per call
constexpr int kNaMaxGrid = 160;                        // CTAs of the scoring kernel
constexpr int kNaMaxDim = DRESD_MAX_DIM;

constexpr size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }
constexpr size_t kOffStatus = 0;
constexpr size_t kOffQhat = align256(sizeof(int));
constexpr size_t kOffQsplit = kOffQhat + align256(sizeof(float) * kNaMaxBatch * kNaMaxDim);
constexpr size_t kOffCand = kOffQsplit + align256((size_t)2 * 2 * kNaMaxBatch * kNaMaxDim);
constexpr size_t kScratchBytes =
    kOffCand + align256(sizeof(unsigned long long) * kNaMaxGrid * kNaMaxBatch * kCandStride);

// The workspace itself.  In host code this name is only a handle for
// cudaGetSymbolAddress(); it is not a device address.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char *g_scratch_ptr[kMaxDevices] = {};        // device address, per device
int g_num_sms[kMaxDevices] = {};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn g_encode = nullptr;                      // resolved in setup_device(), under g_mutex

// Host-side descriptor of the key matrix (no device memory involved).
bool encode_key_map(CUtensorMap *map, const void *base, int dtype, long long rows, int cols, int box_rows)
{
    EncodeTiledFn fn = g_encode;
    if (!fn) return false;
    const size_t eb = dtype == kF32 ? 4 : 2;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * eb};
    cuuint32_t box[2] = {(cuuint32_t)(128 / eb), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMapDataType dt = dtype == kF32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                             : dtype == kF16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                             : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    return fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

dresd_status na_fail(dresd_status st, const char *msg)
{
    set_last_error(msg);            // readable through dresd_last_error()
    return st;
}

// One-time set-up for the current device: resolve the device address of the
// workspace.  Runs on the first call per device.
dresd_status setup_device(int dev, unsigned char **ptr_out, int *sms_out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        unsigned char *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_scratch);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            return na_fail(DRESD_ERR_CUDA, "cudaGetSymbolAddress failed for the static workspace");
        }
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess || sms <= 0) return na_fail(DRESD_ERR_CUDA, "cannot query the SM count");
        if (!g_encode) {
            void *p = nullptr;
            cudaDriverEntryPointQueryResult q;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
                q != cudaDriverEntryPointSuccess)
                return na_fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
            g_encode = reinterpret_cast<EncodeTiledFn>(p);
        }
        g_num_sms[dev] = sms;
        g_scratch_ptr[dev] = ptr;
    }
    *ptr_out = g_scratch_ptr[dev];
    *sms_out = g_num_sms[dev];
    return DRESD_OK;
}

}  // namespace

extern "C" dresd_status dresd_retrieve_noalloc(const void *keys, const int32_t *next_tokens, int64_t N, int d,
                                               dresd_dtype dtype, int stored_len, const void *queries, int B,
                                               int top_n, int draft_len, int32_t *out_ids, float *out_scores,
                                               int32_t *out_tokens, void *stream_v)
{
    if (dtype != DRESD_F32 && dtype != DRESD_F16 && dtype != DRESD_BF16)
        return na_fail(DRESD_ERR_INVALID, "unknown dtype");
    if (N <= 0 || N > kMaxRows) return na_fail(DRESD_ERR_INVALID, "N outside 1..2^31-1024");
    if (d <= 0 || stored_len < 1) return na_fail(DRESD_ERR_INVALID, "bad d or stored_len");
    const size_t eb = dtype == DRESD_F32 ? 4 : 2;
    if (((size_t)d * eb) % 16 != 0) return na_fail(DRESD_ERR_INVALID, "row size is not a multiple of 16 bytes");
    if (!keys || !next_tokens) return na_fail(DRESD_ERR_INVALID, "keys / next_tokens is NULL");
    if (reinterpret_cast<uintptr_t>(keys) % 16 != 0) return na_fail(DRESD_ERR_INVALID, "keys not 16-byte aligned");
    if (B < 0) return na_fail(DRESD_ERR_INVALID, "B is negative");
    if (top_n < 1 || top_n > N) return na_fail(DRESD_ERR_INVALID, "top_n outside 1..N");
    if (draft_len < 1 || draft_len > stored_len) return na_fail(DRESD_ERR_INVALID, "draft_len outside 1..stored_len");
    if (B > kNaMaxBatch)
        return na_fail(DRESD_ERR_UNSUPPORTED, "B exceeds DRESD_NOALLOC_MAX_BATCH: the static workspace holds 8 queries");
    if (top_n > DRESD_MAX_TOP_N) return na_fail(DRESD_ERR_UNSUPPORTED, "top_n exceeds DRESD_MAX_TOP_N");
    if (d > kNaMaxDim) return na_fail(DRESD_ERR_UNSUPPORTED, "d exceeds DRESD_MAX_DIM");
    if (B == 0) return DRESD_OK;
    if (!queries || !out_ids || !out_scores || !out_tokens) return na_fail(DRESD_ERR_INVALID, "NULL buffer");

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return na_fail(DRESD_ERR_CUDA, "cudaGetDevice failed");
    if (dev < 0 || dev >= kMaxDevices) return na_fail(DRESD_ERR_UNSUPPORTED, "device ordinal beyond 63");
    unsigned char *scratch = nullptr;
    int sms = 0;
    dresd_status st = setup_device(dev, &scratch, &sms);
    if (st != DRESD_OK) return st;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int *status = reinterpret_cast<int *>(scratch + kOffStatus);
    unsigned int *gtau = reinterpret_cast<unsigned int *>(scratch + kOffStatus + 128);   // 8 words
    float *qhat = reinterpret_cast<float *>(scratch + kOffQhat);
    void *qsplit = scratch + kOffQsplit;
    unsigned long long *cand = reinterpret_cast<unsigned long long *>(scratch + kOffCand);

    const bool f32 = dtype == DRESD_F32;
    const int dpad = ((d + 63) / 64) * 64;
    const int tile_rows = f32 ? scan_f32_tile_rows(d) : scan_mma_tile_rows(d);
    const int n_tiles = (int)((N + tile_rows - 1) / tile_rows);
    CUtensorMap map;
    if (!encode_key_map(&map, keys, (int)dtype, N, d, f32 ? scan_f32_box_rows(d) : tile_rows))
        return na_fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the key matrix");

    // The workspace keeps the previous call's contents.  Only the status word
    // must start at zero; every other word that is read is written first.
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess)
        return na_fail(DRESD_ERR_CUDA, "cudaMemsetAsync failed");

    const float lo_scale = dtype == DRESD_F16 ? kHiLoScaleF16 : kHiLoScaleBF16;
    PreprocessArgs p{};
    p.queries = queries;
    p.eps_z = 1e-5f;
    p.eps_n = 1e-12f;
    p.B = B;
    p.d_in = d;
    p.d = d;
    p.dtype = (int)dtype;
    p.qhat = qhat;
    p.qsplit = f32 ? nullptr : qsplit;
    p.dpad = dpad;
    p.rows = kNaMaxBatch;
    p.lo_scale = lo_scale;
    p.gtau = gtau;
    if (launch_preprocess(p, stream) != cudaSuccess) return na_fail(DRESD_ERR_CUDA, "preprocess launch failed");

    int grid = sms < kNaMaxGrid ? sms : kNaMaxGrid;
    if (grid > n_tiles) grid = n_tiles;
    const int qpl = f32 ? scan_f32_queries_per_launch(d, B) : scan_mma_queries_per_launch(d, B);
    for (int q0 = 0; q0 < B; q0 += qpl) {
        ScanArgs a{};
        a.N = N;
        a.d = d;
        a.dpad = dpad;
        a.dtype = (int)dtype;
        a.n_tiles = n_tiles;
        a.B = B - q0 < qpl ? B - q0 : qpl;
        a.top_n = top_n;
        a.qhat = qhat + (size_t)q0 * d;
        a.qsplit = f32 ? nullptr : static_cast<const unsigned char *>(qsplit) + (size_t)2 * q0 * dpad * 2;
        a.lo_inv_scale = 1.0f / lo_scale;
        a.cand = cand + (size_t)q0 * kCandStride;
        a.cand_batch = B;
        a.status = status;
        a.gtau = gtau + q0;
        cudaError_t e = f32 ? launch_scan_f32(map, a, grid, stream) : launch_scan_mma(map, a, grid, stream);
        if (e != cudaSuccess) return na_fail(DRESD_ERR_CUDA, "scan launch failed");
    }
    if (launch_merge_gather(cand, grid, B, top_n, out_ids, out_scores, next_tokens, stored_len, N, draft_len,
                            out_tokens, stream) != cudaSuccess)
        return na_fail(DRESD_ERR_CUDA, "merge/gather launch failed");
    return DRESD_OK;
}

// The status word of the static workspace: the scoring kernels' bounded waits record a give-up
// there.  Reading it needs a 4-byte copy into the caller's stack and nothing else.
extern "C" dresd_status dresd_noalloc_status(void *stream_v)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return na_fail(DRESD_ERR_CUDA, "cudaGetDevice failed");
    if (dev < 0 || dev >= kMaxDevices) return na_fail(DRESD_ERR_UNSUPPORTED, "device ordinal beyond 63");
    unsigned char *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        scratch = g_scratch_ptr[dev];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    if (!scratch) {                                     // no call was made on this device yet
        if (cudaStreamSynchronize(stream) != cudaSuccess) return na_fail(DRESD_ERR_CUDA, "stream synchronize failed");
        return DRESD_OK;
    }
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, scratch + kOffStatus, sizeof(int), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return na_fail(DRESD_ERR_CUDA, "status read failed");
    if (word != 0) {
        cudaMemsetAsync(scratch + kOffStatus, 0, sizeof(int), stream);
        return na_fail(DRESD_ERR_TIMEOUT, "a device-side wait expired");
    }
    return DRESD_OK;
}

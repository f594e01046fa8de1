// C ABI of the retrieval library: store object, argument validation, TMA
// descriptors, workspace, and the launch chain K1 -> K2+K3 -> K4 -> K5.
// See include/dresd.h for the contract of every entry point.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>
#include <new>

#include "../../include/dresd.h"
#include "internal.h"

using namespace dresd;

namespace {

thread_local char g_err[512] = "";

dresd_status fail(dresd_status st, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return st;
}
dresd_status fail_cuda(cudaError_t e, const char *what)
{
    return fail(DRESD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

constexpr uint32_t kMagic = 0xD2E5D001u;
constexpr int kProbeAuto = 1;        // default: the stride follows the store (about four probe tiles per CTA)
constexpr float kEpsNorm = 1e-12f;   // epsilon of Eq. 2 (the paper leaves it open)

bool is_device_ptr(const void *p)
{
    if (!p) return false;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

size_t elem_bytes(int dtype) { return dtype == kF32 ? 4 : 2; }

// Device-side address of a page-locked host buffer that the device can reach, else null.
void *mapped_device_ptr(const void *host)
{
    cudaPointerAttributes at{};
    if (!host || cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// 2-D map over a row-major [rows][cols] matrix; box = one 128-byte swizzle row
// wide, box_rows tall; out-of-range elements read as zero.
bool make_map(CUtensorMap *map, const void *base, int dtype, long long rows, int cols, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const size_t eb = elem_bytes(dtype);
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * eb};
    cuuint32_t box[2] = {(cuuint32_t)(128 / eb), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMapDataType dt = dtype == kF32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                             : dtype == kF16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                             : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUresult r = fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

void dresd::set_last_error(const char *msg) { snprintf(g_err, sizeof g_err, "%s", msg ? msg : ""); }

struct dresd_store {
    uint32_t magic;
    int device;
    int num_sms;
    // datastore (borrowed)
    const void *keys;
    const int32_t *next_tokens;
    long long N;
    int d, dpad, dtype, stored_len;
    // preprocessing (borrowed)
    int d_in;
    const float *mean, *var, *pca_mean;
    const void *W;
    float eps_z;
    // workspace (owned)
    float *qhat;                 // [kMaxBatch][d]
    void *qsplit;                // [2*kMaxBatch][dpad] 16-bit
    unsigned long long *cand;    // [max_grid][kMaxBatch][kCandStride]
    int *status;                 // device status word
    unsigned int *gtau;          // [kMaxBatch] grid-wide filter words
    int32_t *first_col;          // [N] first stored token of every key; allocated on request
    int32_t *win_start;          // [win_vocab + 1] rows of every first token (sorted stores); on request
    int win_vocab, opt_windows;
    int max_grid;
    // staging for dresd_retrieve_host (owned, device)
    void *q_stage;
    size_t q_stage_bytes;
    int32_t *ids_dev;
    float *scores_dev;
    int32_t *tokens_dev;
    size_t tokens_dev_elems;
    // streaming-kernel geometry
    CUtensorMap map_stream;
    int tile_rows, n_tiles;
    // tensor-core kernel geometry (16-bit keys): 128-row key tiles, query operand maps
    CUtensorMap map_umma;
    CUtensorMap map_q[4];        // box rows 16 / 32 / 64 / 128 over qsplit
    // options / bookkeeping
    int opt_path, opt_grid, opt_probe, opt_wait_ms, opt_lose_stage, opt_no_select, opt_keys_as_m, opt_pack2, opt_merged, opt_round_per_tile, opt_no_fast_reject, opt_epi_warps, opt_merge_level;
    double last_key_passes;      // passes over the key matrix in the last call (a probe pass counts 1/stride)
    const void *k8;              // 8-bit (E4M3) copy of the keys, borrowed; null = none attached
    void *qsplit8;               // [2 * kMaxBatch][dpad8] 8-bit query operand
    int dpad8;                   // d rounded up to 128 bytes
    CUtensorMap map_k8, map_q8[4];
    CUtensorMap map_k8p;         // d = 64: the 8-bit copy as N/2 rows of two keys (128 bytes)
    int k8_packable;
    CUtensorMap map_k16p;        // 16-bit keys, d = 32, even N: the store as N/2 rows of two keys (128 bytes)
    int k16_packable;
    int prof_stride, prof_calls;
    float *proj_ws;              // partial products of the split projection (allocated with W)
    size_t proj_ws_bytes;
    cudaStream_t last_stream;
    int last_launches;
    // optional timing of the scoring kernel (option "profile")
    cudaEvent_t *prof_events;    // [2 * prof_cap]: start/stop pairs
    int prof_cap, prof_count;
};

namespace {

bool valid(const dresd_store *s) { return s && s->magic == kMagic; }

void free_store(dresd_store *s)
{
    if (!s) return;
    cudaFree(s->qhat);
    cudaFree(s->qsplit);
    cudaFree(s->cand);
    cudaFree(s->status);
    cudaFree(s->gtau);
    cudaFree(s->first_col);
    cudaFree(s->win_start);
    cudaFree(s->q_stage);
    cudaFree(s->proj_ws);
    cudaFree(s->qsplit8);
    cudaFree(s->ids_dev);
    cudaFree(s->scores_dev);
    cudaFree(s->tokens_dev);
    for (int i = 0; i < 2 * s->prof_cap; ++i) cudaEventDestroy(s->prof_events[i]);
    delete[] s->prof_events;
    s->magic = 0;
    delete s;
}

// A store launches on the device it was created on (its workspace and descriptors live there).
dresd_status check_device(const dresd_store *s)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != s->device)
        return fail(DRESD_ERR_INVALID, "the store belongs to device %d; the current device is %d", s->device, dev);
    return DRESD_OK;
}

dresd_status check_retrieve_args(const dresd_store *s, const void *queries, int B, int top_n,
                                 int draft_len, const void *ids, const void *scores,
                                 const void *tokens, bool device_ptrs)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    if (dresd_status ds = check_device(s)) return ds;
    if (B < 0) return fail(DRESD_ERR_INVALID, "B = %d is negative", B);
    if (top_n < 1 || top_n > s->N) return fail(DRESD_ERR_INVALID, "top_n = %d outside 1..N", top_n);
    if (draft_len < 1 || draft_len > s->stored_len)
        return fail(DRESD_ERR_INVALID, "draft_len = %d outside 1..stored_len (%d)", draft_len, s->stored_len);
    if (B > DRESD_MAX_BATCH) return fail(DRESD_ERR_UNSUPPORTED, "B = %d exceeds DRESD_MAX_BATCH", B);
    if (top_n > DRESD_MAX_TOP_N) return fail(DRESD_ERR_UNSUPPORTED, "top_n = %d exceeds DRESD_MAX_TOP_N", top_n);
    if (B == 0) return DRESD_OK;
    if (!queries || !ids || !scores || !tokens) return fail(DRESD_ERR_INVALID, "NULL buffer");
    if (device_ptrs && (!is_device_ptr(queries) || !is_device_ptr(ids) || !is_device_ptr(scores) ||
                        !is_device_ptr(tokens)))
        return fail(DRESD_ERR_INVALID, "queries/out_* must be device pointers");
    return DRESD_OK;
}

// K1 for B queries into the store's workspace.
// quantised: 0 = no, 1 = also write the 8-bit query terms, 2 = in the packed (two keys per row) layout
dresd_status run_preprocess(dresd_store *s, const void *queries, int B, int rows, cudaStream_t stream,
                            int split_blocked = 0, int quantised = 0)
{
    PreprocessArgs p{};
    p.queries = queries;
    p.mean = s->mean;
    p.var = s->var;
    p.W = s->W;
    p.pca_mean = s->pca_mean;
    p.eps_z = s->eps_z;
    p.eps_n = kEpsNorm;
    p.B = B;
    p.d_in = s->d_in;
    p.d = s->d;
    p.dtype = s->dtype;
    p.qhat = s->qhat;
    p.qsplit = s->dtype == kF32 ? nullptr : s->qsplit;
    p.dpad = s->dpad;
    p.rows = rows;                   // operand rows beyond B are written as zeros
    p.lo_scale = s->dtype == kF16 ? kHiLoScaleF16 : kHiLoScaleBF16;
    p.gtau = s->gtau;
    p.split_blocked = split_blocked;
    if (quantised) {
        p.qsplit8 = static_cast<uint8_t *>(s->qsplit8);
        p.dpad8 = s->dpad8;
        p.pack2 = quantised == 2;
    }
    if (s->W && s->proj_ws && reinterpret_cast<uintptr_t>(s->W) % 16 == 0) {     // 16-byte loads of W rows
        preprocess_split_plan(s->d_in, s->d, B, (int)elem_bytes(s->dtype), s->proj_ws_bytes, &p.slices, &p.rows_per_slice);
        if (p.slices > 0) p.partial = s->proj_ws;
    }
    cudaError_t e = launch_preprocess(p, stream);
    if (e != cudaSuccess) return fail_cuda(e, "preprocess launch");
    s->last_launches += p.partial ? 2 : 1;
    return DRESD_OK;
}

dresd_status run_retrieve(dresd_store *s, const void *queries, int B, int top_n, int draft_len,
                          int32_t *out_ids, float *out_scores, int32_t *out_tokens, cudaStream_t stream,
                          const int32_t *first_tokens = nullptr, int quantised_m = 0)
{
    // quantised_m > 0: candidates by approximate score over the 8-bit copy of the keys (the same
    // tcgen05 kernel, other instruction kind), then exact re-ranking of the quantised_m best
    const bool q8 = quantised_m > 0;
    // 64-element keys are 64 bytes in the 8-bit copy: two per 128-byte row, two column pairs per query
    const bool pack8 = q8 && s->k8_packable && B <= kMaxBatch / 2 && s->opt_pack2;
    // 32-element 16-bit keys are 64 bytes as well: the same two-keys-per-row scan for up to 16 queries
    // (more run the form with one accumulator column per query)
    const bool pack16 = !q8 && s->dtype != kF32 && s->opt_path != 1 && s->k16_packable && B <= 16 && s->opt_pack2;
    const bool pack2 = pack8 || pack16;
    s->last_stream = stream;
    s->last_launches = 0;
    s->last_key_passes = 0.0;
    const bool f32 = s->dtype == kF32;
    // 16-bit keys: the tcgen05 kernel serves any batch in one pass over the keys and is
    // the fastest at every measured shape (7.1-7.2 TB/s at batch 1 for d = 64 and 256
    // against 6.7-6.8 for the streaming mma.sync kernel), so it is the default; the
    // streaming kernel stays available as "scan_path" 1 and serves the allocation-free call.
    const bool umma = q8 || (!f32 && s->opt_path != 1);
    // sorted store with an index: the kernel with the keys as M scans the queries' token windows only
    const bool windows = umma && first_tokens && s->win_start && s->opt_windows;
    const int keys_as_m = (q8 || s->opt_keys_as_m || windows) ? 1 : 0;
    // the kernel with the keys as the N operand reads hi and lo of a query from one TMEM fragment;
    // its operand always has 128 rows (64 hi, 64 lo), whatever the batch
    const int blocked = umma && !keys_as_m && scan_ummat_eligible(s->d, B);
    // more than 16 queries on the other widths: one accumulator column per query (half the epilogue's work)
    const int merged = umma && !q8 && !blocked && !pack16 && s->opt_merged != 2 &&
                       (s->opt_merged == 1 ? B > 16 : scan_umma_merged_eligible(s->d, B, s->dtype));
    const int op_rows = !umma ? 0 : blocked ? 2 * kMaxBatch : scan_umma_operand_rows(pack2 ? 2 * B : B);
    // one CTA per operand query: two operand rows each, four in the packed 8-bit layout
    const int pre_rows = pack2 ? op_rows / 4 : umma ? op_rows / 2 : ((B + 7) / 8) * 8;
    // operand layouts (PreprocessArgs::split_blocked): the tcgen05 kernel with the keys as M takes the hi rows of all
    // queries first, then the lo rows (4); its one-column form both scaled (2); 32-element keys two per row (3);
    // the kernel with the keys as N 16-row blocks (1); the streaming kernel and the 8-bit search pairs (0)
    const int layout = pack16 ? 3 : merged ? 2 : blocked ? 1 : (umma && !q8) ? 4 : 0;
    dresd_status st = run_preprocess(s, queries, B, pre_rows, stream, layout, pack8 ? 2 : q8 ? 1 : 0);
    if (st != DRESD_OK) return st;

    // the 8-bit store is scanned as rows of d/2 two-byte units (packed: N/2 rows of 64 units)
    const int scan_d = pack2 ? 64 : q8 ? s->d / 2 : s->d;
    const long long scan_rows = pack2 ? s->N / 2 : s->N;
    const int umma_rows = umma ? scan_umma_tile_rows(scan_d, pack2 ? 2 * B : B, keys_as_m, merged) : 1;
    const int n_tiles = umma ? (int)((scan_rows + umma_rows - 1) / umma_rows) : s->n_tiles;
    int grid = s->opt_grid > 0 ? s->opt_grid : s->num_sms;
    if (grid > s->max_grid) grid = s->max_grid;
    if (grid > n_tiles) grid = n_tiles;

    const int qpl = umma ? B : f32 ? scan_f32_queries_per_launch(s->d, B) : scan_mma_queries_per_launch(s->d, B);
    const float lo_scale = s->dtype == kF16 ? kHiLoScaleF16 : kHiLoScaleBF16;
    // timing events sit between the kernels of a call and so hold up their overlap: with a stride only
    // every stride-th call of the armed window carries them
    const bool prof = s->prof_count < s->prof_cap && (s->prof_calls++ % (s->prof_stride > 0 ? s->prof_stride : 1)) == 0;
    if (prof) cudaEventRecord(s->prof_events[2 * s->prof_count], stream);
    if (umma) {
        ScanArgs a{};
        a.N = scan_rows;
        a.pack2 = pack2 ? 1 : 0;
        a.d = scan_d;
        a.dpad = q8 ? s->dpad8 / 2 : s->dpad;
        a.dtype = q8 ? kE4M3 : s->dtype;
        a.n_tiles = n_tiles;
        a.B = B;
        a.top_n = q8 ? quantised_m : top_n;
        a.lo_inv_scale = q8 ? 1.0f / 16.0f : 1.0f / lo_scale;
        a.cand = s->cand;
        a.cand_batch = B;
        a.status = s->status;
        a.gtau = s->gtau;
        a.no_select = s->opt_no_select;
        a.keys_as_m = keys_as_m;
        a.merged = merged;
        a.round_per_tile = s->opt_round_per_tile;
        a.no_fast_reject = s->opt_no_fast_reject;
        a.epi_warps = s->opt_epi_warps;
        a.merge_level = s->opt_merge_level;
        a.wait_cycles = (long long)s->opt_wait_ms * 2000000LL;     // ~2 GHz
        a.debug_lose_stage = s->opt_lose_stage;
        if (windows) {
            a.win_start = s->win_start;
            a.win_vocab = s->win_vocab;
        }
        const CUtensorMap &kmap = pack8 ? s->map_k8p : pack16 ? s->map_k16p : q8 ? s->map_k8 : s->map_umma;
        const CUtensorMap *qmaps = q8 ? s->map_q8 : s->map_q;
        const int sel_n = a.top_n;
        a.first_col = first_tokens ? s->first_col : nullptr;
        a.want_first = first_tokens;
        const int mi = op_rows == 16 ? 0 : op_rows == 32 ? 1 : op_rows == 64 ? 2 : 3;
        cudaError_t e = cudaSuccess;
        // Large batches on large stores: a probe pass over every pstride-th tile first.  Its
        // n-th best score per query seeds the grid-wide filter, so that the full pass
        // queues ~pstride n survivors per query GPU-wide instead of ~n ln(rows/n) per CTA.
        // The filter only rejects rows that cannot be in the result.
        int pstride = s->opt_probe;
        if (pstride == kProbeAuto) {
            // The full pass queues ~pstride n survivors per query, the probe pass costs 1/pstride of a full
            // pass plus its fixed part (launch, set-up, one tile's latency): the best stride falls with
            // sqrt(B n) -- 64 measured best at 64 queries x top-32, 128-256 at top-10 -- and a small
            // store still gets one probe tile per CTA.
            const double t = 2900.0 / sqrt((double)B * sel_n);
            pstride = t < 64.0 ? 64 : t > 256.0 ? 256 : (int)t;
            // one best per 128 rows and CTA must fit the CTA's queue of 32 (the cheap form of the probe pass)
            const long long fit = ((long long)n_tiles * (umma_rows / 128) + 32LL * grid - 1) / (32LL * grid);
            if (pstride < fit) pstride = (int)fit;
            if ((long long)pstride * grid > n_tiles) pstride = n_tiles / grid;
            if (pstride < 2) pstride = 0;
        }
        if (pstride > 1 && !s->opt_no_select && B * sel_n >= 256 && n_tiles >= pstride * grid) {
            ScanArgs pa = a;
            pa.tile_stride = pstride;
            pa.n_tiles = (n_tiles + pstride - 1) / pstride;
            pa.probe_max = (long long)pa.n_tiles * (umma_rows / 128) <= 32LL * grid;   // the bests fit a queue
            int pgrid = grid < pa.n_tiles ? grid : pa.n_tiles;
            e = launch_scan_umma(kmap, qmaps[mi], pa, pgrid, stream);
            if (e == cudaSuccess) e = launch_merge_tau(s->cand, pgrid, B, sel_n, s->gtau, stream);
            if (e != cudaSuccess) return fail_cuda(e, "probe launch");
            s->last_launches += 2;
            s->last_key_passes += 1.0 / pstride;
        }
        e = launch_scan_umma(kmap, qmaps[mi], a, grid, stream);
        if (e != cudaSuccess) return fail_cuda(e, "scan launch");
        s->last_launches += 1;
        s->last_key_passes += 1.0;
    }
    for (int q0 = 0; q0 < B && !umma; q0 += qpl) {
        ScanArgs a{};
        a.N = s->N;
        a.d = s->d;
        a.dpad = s->dpad;
        a.dtype = s->dtype;
        a.n_tiles = s->n_tiles;
        a.B = B - q0 < qpl ? B - q0 : qpl;
        a.top_n = top_n;
        a.qhat = s->qhat + (size_t)q0 * s->d;
        a.qsplit = f32 ? nullptr
                       : static_cast<const uint8_t *>(s->qsplit) + (size_t)2 * q0 * s->dpad * 2;
        a.lo_inv_scale = 1.0f / lo_scale;
        a.cand = s->cand + (size_t)q0 * kCandStride;
        a.cand_batch = B;
        a.status = s->status;
        a.gtau = s->gtau + q0;
        a.wait_cycles = (long long)s->opt_wait_ms * 2000000LL;     // ~2 GHz
        a.debug_lose_stage = s->opt_lose_stage;
        a.first_col = first_tokens ? s->first_col : nullptr;
        a.want_first = first_tokens ? first_tokens + q0 : nullptr;
        cudaError_t e = f32 ? launch_scan_f32(s->map_stream, a, grid, stream)
                            : launch_scan_mma(s->map_stream, a, grid, stream);
        if (e != cudaSuccess) return fail_cuda(e, "scan launch");
        s->last_launches += 1;
        s->last_key_passes += 1.0;
    }
    if (prof) {
        cudaEventRecord(s->prof_events[2 * s->prof_count + 1], stream);
        s->prof_count += 1;
    }
    if (q8) {
        // fold the approximate lists, score the m survivors exactly, sort, gather: one launch
        cudaError_t e = launch_merge_rerank(s->cand, grid, B, s->keys, s->dtype, s->d, s->N, s->qhat, quantised_m, top_n,
                                            pack8 && (s->N & 1) ? s->N - 1 : -1, first_tokens, s->next_tokens, s->stored_len,
                                            draft_len, out_ids, out_scores, out_tokens, stream);
        if (e != cudaSuccess) return fail_cuda(e, "merge / re-rank launch");
        s->last_launches += 1;
        return DRESD_OK;
    }
    cudaError_t e = launch_merge_gather(s->cand, grid, B, top_n, out_ids, out_scores, s->next_tokens, s->stored_len,
                                        s->N, draft_len, out_tokens, stream, s->status);
    if (e != cudaSuccess) return fail_cuda(e, "merge/gather launch");
    s->last_launches += 1;
    return DRESD_OK;
}

}  // namespace

namespace {
// Scratch of the datastore-building calls (the split copy of W, partial sums): kept per device
// between calls and only ever grown, so that building a datastore chunk by chunk does not
// allocate and free on every call.  Callers hold g_scratch_mutex until their work has finished.
constexpr int kScratchDevices = 64;
std::mutex g_scratch_mutex;
uint8_t *g_scratch_ptr[kScratchDevices] = {};
size_t g_scratch_size[kScratchDevices] = {};

std::atomic<int> g_build_pairs{1};      // dresd_build_keys on CTA pairs (cta_group::2); 0 = one CTA per tile
std::atomic<int> g_build_wait_ms{0};    // bound of dresd_build_keys' device-side waits, 0 = default
std::atomic<int> g_build_lose_stage{0}; // test hook: the first CTA (pair) never receives stage (value-1)

uint8_t *device_scratch(int dev, size_t need)
{
    if (g_scratch_size[dev] < need) {
        cudaFree(g_scratch_ptr[dev]);
        g_scratch_ptr[dev] = nullptr;
        g_scratch_size[dev] = 0;
        if (cudaMalloc(&g_scratch_ptr[dev], need) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        g_scratch_size[dev] = need;
    }
    return g_scratch_ptr[dev];
}

}  // namespace

extern "C" {

dresd_status dresd_store_create(const void *keys, const int32_t *next_tokens, int64_t N, int d,
                                dresd_dtype dtype, int stored_len, dresd_store **out_store)
{
    if (!out_store) return fail(DRESD_ERR_INVALID, "out_store is NULL");
    *out_store = nullptr;
    if (dtype != DRESD_F32 && dtype != DRESD_F16 && dtype != DRESD_BF16)
        return fail(DRESD_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (N <= 0 || N > kMaxRows) return fail(DRESD_ERR_INVALID, "N = %lld outside 1..2^31-1024", (long long)N);
    if (d <= 0) return fail(DRESD_ERR_INVALID, "d = %d", d);
    if (stored_len < 1) return fail(DRESD_ERR_INVALID, "stored_len = %d", stored_len);
    const size_t eb = elem_bytes((int)dtype);
    if (((size_t)d * eb) % 16 != 0)
        return fail(DRESD_ERR_INVALID, "row size %zu bytes is not a multiple of 16", (size_t)d * eb);
    if (!keys || !next_tokens) return fail(DRESD_ERR_INVALID, "keys / next_tokens is NULL");
    if (reinterpret_cast<uintptr_t>(keys) % 16 != 0) return fail(DRESD_ERR_INVALID, "keys not 16-byte aligned");
    if (d > DRESD_MAX_DIM) return fail(DRESD_ERR_UNSUPPORTED, "d = %d exceeds DRESD_MAX_DIM", d);

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDevice");
    if (!is_device_ptr(keys) || !is_device_ptr(next_tokens))
        return fail(DRESD_ERR_INVALID, "keys / next_tokens must be device pointers");
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDeviceProperties");
    if (prop.major != 10) return fail(DRESD_ERR_UNSUPPORTED, "device is sm_%d%d; this library is built for sm_100a", prop.major, prop.minor);

    dresd_store *s = new (std::nothrow) dresd_store();
    if (!s) return fail(DRESD_ERR_ALLOC, "host allocation failed");
    memset(s, 0, sizeof *s);
    s->magic = kMagic;
    s->device = dev;
    s->num_sms = prop.multiProcessorCount;
    s->keys = keys;
    s->next_tokens = next_tokens;
    s->N = N;
    s->d = d;
    s->dpad = ((d + 63) / 64) * 64;
    s->dtype = (int)dtype;
    s->stored_len = stored_len;
    s->d_in = d;
    s->eps_z = 1e-5f;
    s->max_grid = 2 * s->num_sms;
    s->opt_probe = kProbeAuto;
    s->opt_pack2 = 1;
    s->opt_windows = 1;

    s->tile_rows = dtype == DRESD_F32 ? scan_f32_tile_rows(d) : scan_mma_tile_rows(d);
    s->n_tiles = (int)((N + s->tile_rows - 1) / s->tile_rows);
    if (!make_map(&s->map_stream, keys, s->dtype, N, d, dtype == DRESD_F32 ? scan_f32_box_rows(d) : s->tile_rows)) {
        free_store(s);
        return fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the key matrix");
    }

    bool ok = cudaMalloc(&s->qhat, sizeof(float) * kMaxBatch * (size_t)d) == cudaSuccess &&
              cudaMalloc(&s->qsplit, (size_t)2 * 2 * kMaxBatch * s->dpad) == cudaSuccess &&
              cudaMalloc(&s->cand, sizeof(unsigned long long) * (size_t)s->max_grid * kMaxBatch * kCandStride) == cudaSuccess &&
              cudaMalloc(&s->status, sizeof(int)) == cudaSuccess &&
              cudaMalloc(&s->gtau, sizeof(unsigned int) * kMaxBatch) == cudaSuccess &&
              cudaMalloc(&s->ids_dev, sizeof(int32_t) * kMaxBatch * kMaxTopN) == cudaSuccess &&
              cudaMalloc(&s->scores_dev, sizeof(float) * kMaxBatch * kMaxTopN) == cudaSuccess;
    s->tokens_dev_elems = (size_t)kMaxBatch * kMaxTopN * stored_len;
    ok = ok && cudaMalloc(&s->tokens_dev, sizeof(int32_t) * s->tokens_dev_elems) == cudaSuccess;
    if (ok && dtype != DRESD_F32) {
        bool mok = make_map(&s->map_umma, keys, s->dtype, N, d, 128);
        for (int i = 0; i < 4; ++i)
            mok = mok && make_map(&s->map_q[i], s->qsplit, s->dtype, 2 * kMaxBatch, s->dpad, 16 << i);
        // 32-element keys are 64 bytes: an even-sized store is also seen as N/2 rows of two keys
        if (mok && d == 32 && N >= 2 && (N & 1) == 0) {
            mok = make_map(&s->map_k16p, keys, s->dtype, N / 2, 64, 128);
            s->k16_packable = mok ? 1 : 0;
        }
        if (!mok) {
            free_store(s);
            return fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the tensor-core path");
        }
    }
    s->q_stage_bytes = (size_t)kMaxBatch * d * eb;
    ok = ok && cudaMalloc(&s->q_stage, s->q_stage_bytes) == cudaSuccess;
    ok = ok && cudaMemset(s->status, 0, sizeof(int)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_store(s);
        return fail(DRESD_ERR_ALLOC, "workspace allocation failed");
    }
    *out_store = s;
    return DRESD_OK;
}

dresd_status dresd_store_set_preprocess(dresd_store *s, int d_in, const float *mean, const float *var,
                                        float eps_z, const void *W, const float *pca_mean)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    if (d_in <= 0) return fail(DRESD_ERR_INVALID, "d_in = %d", d_in);
    if ((mean == nullptr) != (var == nullptr)) return fail(DRESD_ERR_INVALID, "mean and var go together");
    if (!W && d_in != s->d) return fail(DRESD_ERR_INVALID, "without W, d_in must equal d");
    if (pca_mean && !W) return fail(DRESD_ERR_INVALID, "pca_mean needs W");
    if (!(eps_z >= 0.f)) return fail(DRESD_ERR_INVALID, "eps_z must be >= 0");
    if ((mean && !is_device_ptr(mean)) || (var && !is_device_ptr(var)) || (W && !is_device_ptr(W)) ||
        (pca_mean && !is_device_ptr(pca_mean)))
        return fail(DRESD_ERR_INVALID, "mean/var/W/pca_mean must be device pointers");
    if (d_in > 16384) return fail(DRESD_ERR_UNSUPPORTED, "d_in = %d exceeds 16384", d_in);
    const size_t need = (size_t)kMaxBatch * d_in * elem_bytes(s->dtype);
    if (need > s->q_stage_bytes) {
        void *p = nullptr;
        if (cudaMalloc(&p, need) != cudaSuccess) {
            cudaGetLastError();
            return fail(DRESD_ERR_ALLOC, "staging allocation failed");
        }
        cudaFree(s->q_stage);
        s->q_stage = p;
        s->q_stage_bytes = need;
    }
    if (W && !s->proj_ws) {
        // workspace of the split projection; without it every query's CTA walks all of W (slow, not wrong)
        const size_t bytes = (size_t)8 << 20;
        void *p = nullptr;
        if (cudaMalloc(&p, bytes) == cudaSuccess) {
            s->proj_ws = static_cast<float *>(p);
            s->proj_ws_bytes = bytes;
        } else {
            cudaGetLastError();
        }
    }
    s->d_in = d_in;
    s->mean = mean;
    s->var = var;
    s->eps_z = eps_z;
    s->W = W;
    s->pca_mean = pca_mean;
    return DRESD_OK;
}

dresd_status dresd_retrieve(dresd_store *s, const void *queries, int B, int top_n, int draft_len,
                            int32_t *out_ids, float *out_scores, int32_t *out_tokens, void *stream)
{
    dresd_status st = check_retrieve_args(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens, true);
    if (st != DRESD_OK || B == 0) return st;
    return run_retrieve(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens,
                        static_cast<cudaStream_t>(stream));
}

dresd_status dresd_retrieve_host(dresd_store *s, const void *queries_host, int B, int top_n, int draft_len,
                                 int32_t *out_ids_host, float *out_scores_host, int32_t *out_tokens_host,
                                 void *stream_v)
{
    dresd_status st = check_retrieve_args(s, queries_host, B, top_n, draft_len, out_ids_host,
                                          out_scores_host, out_tokens_host, false);
    if (st != DRESD_OK || B == 0) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t qbytes = (size_t)B * s->d_in * elem_bytes(s->dtype);
    const size_t n = (size_t)B * top_n;
    int dev_status = 0;
    cudaError_t e;
    // Pinned (page-locked, mapped) host buffers are reachable from the device: the kernels then
    // read the queries and write the results across the bus themselves, and no copy is enqueued
    // around them.  Any pageable buffer sends the call through staging copies instead.
    const void *dq = mapped_device_ptr(queries_host);
    int32_t *dids = static_cast<int32_t *>(mapped_device_ptr(out_ids_host));
    float *dsc = static_cast<float *>(mapped_device_ptr(out_scores_host));
    int32_t *dtok = static_cast<int32_t *>(mapped_device_ptr(out_tokens_host));
    if (dq && dids && dsc && dtok) {
        st = run_retrieve(s, dq, B, top_n, draft_len, dids, dsc, dtok, stream);
        if (st != DRESD_OK) return st;
        e = cudaMemcpyAsync(&dev_status, s->status, sizeof(int), cudaMemcpyDeviceToHost, stream);
    } else {
        e = cudaMemcpyAsync(s->q_stage, queries_host, qbytes, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return fail_cuda(e, "query upload");
        st = run_retrieve(s, s->q_stage, B, top_n, draft_len, s->ids_dev, s->scores_dev, s->tokens_dev, stream);
        if (st != DRESD_OK) return st;
        e = cudaMemcpyAsync(out_ids_host, s->ids_dev, n * sizeof(int32_t), cudaMemcpyDeviceToHost, stream);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(out_scores_host, s->scores_dev, n * sizeof(float), cudaMemcpyDeviceToHost, stream);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(out_tokens_host, s->tokens_dev, n * draft_len * sizeof(int32_t),
                                cudaMemcpyDeviceToHost, stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(&dev_status, s->status, sizeof(int), cudaMemcpyDeviceToHost, stream);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return fail_cuda(e, "result download");
    if (dev_status != 0) {
        cudaMemsetAsync(s->status, 0, sizeof(int), stream);
        return fail(DRESD_ERR_TIMEOUT, "a device-side wait expired");
    }
    return DRESD_OK;
}

dresd_status dresd_store_enable_first_token_filter(dresd_store *s, void *stream_v)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    if (s->first_col) return DRESD_OK;
    if (dresd_status ds = check_device(s)) return ds;
    int32_t *col = nullptr;
    if (cudaMalloc(&col, sizeof(int32_t) * (size_t)s->N) != cudaSuccess) {
        cudaGetLastError();
        return fail(DRESD_ERR_ALLOC, "allocation of the first-token column (%lld bytes) failed", 4LL * s->N);
    }
    cudaError_t e = launch_extract_first(s->next_tokens, s->stored_len, s->N, col, static_cast<cudaStream_t>(stream_v));
    if (e != cudaSuccess) {
        cudaFree(col);
        return fail_cuda(e, "first-token column launch");
    }
    s->first_col = col;
    return DRESD_OK;
}

dresd_status dresd_store_index_first_tokens(dresd_store *s, void *stream_v)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    if (s->win_start) return DRESD_OK;
    dresd_status st = dresd_store_enable_first_token_filter(s, stream_v);
    if (st != DRESD_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    // sortedness and the largest token, through the status word's neighbour: a set-up call may synchronise
    int *flag = nullptr;
    if (cudaMalloc(&flag, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return fail(DRESD_ERR_ALLOC, "allocation failed");
    }
    int word = 0, last = 0;
    cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), stream);
    if (e == cudaSuccess) e = launch_check_sorted(s->first_col, s->N, flag, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&word, flag, sizeof(int), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(&last, s->first_col + (s->N - 1), sizeof(int), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    cudaFree(flag);
    if (e != cudaSuccess) return fail_cuda(e, "first-token order check");
    if (word & 2) return fail(DRESD_ERR_INVALID, "a stored first token is negative");
    if (word & 1) return fail(DRESD_ERR_INVALID, "the rows are not sorted by first stored token");
    if (last >= (1 << 24)) return fail(DRESD_ERR_UNSUPPORTED, "largest first token %d exceeds 2^24 - 1", last);
    const int vocab = last + 1;
    int32_t *ws = nullptr;
    if (cudaMalloc(&ws, sizeof(int32_t) * ((size_t)vocab + 1)) != cudaSuccess) {
        cudaGetLastError();
        return fail(DRESD_ERR_ALLOC, "allocation of the window table (%d entries) failed", vocab + 1);
    }
    e = launch_build_windows(s->first_col, s->N, vocab, ws, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) {
        cudaFree(ws);
        return fail_cuda(e, "window table launch");
    }
    s->win_start = ws;
    s->win_vocab = vocab;
    return DRESD_OK;
}

dresd_status dresd_retrieve_filtered(dresd_store *s, const void *queries, const int32_t *first_tokens, int B,
                                     int top_n, int draft_len, int32_t *out_ids, float *out_scores,
                                     int32_t *out_tokens, void *stream)
{
    dresd_status st = check_retrieve_args(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens, true);
    if (st != DRESD_OK || B == 0) return st;
    if (!first_tokens)
        return run_retrieve(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens,
                            static_cast<cudaStream_t>(stream));
    if (!is_device_ptr(first_tokens)) return fail(DRESD_ERR_INVALID, "first_tokens must be a device pointer");
    if (!s->first_col)
        return fail(DRESD_ERR_INVALID, "call dresd_store_enable_first_token_filter() on this store first");
    return run_retrieve(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens,
                        static_cast<cudaStream_t>(stream), first_tokens);
}

dresd_status dresd_preprocess(dresd_store *s, const void *queries, int B, float *out_qhat, void *stream_v)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    if (B < 0) return fail(DRESD_ERR_INVALID, "B = %d is negative", B);
    if (B > DRESD_MAX_BATCH) return fail(DRESD_ERR_UNSUPPORTED, "B = %d exceeds DRESD_MAX_BATCH", B);
    if (B == 0) return DRESD_OK;
    if (dresd_status ds = check_device(s)) return ds;
    if (!is_device_ptr(queries) || !is_device_ptr(out_qhat))
        return fail(DRESD_ERR_INVALID, "queries/out_qhat must be device pointers");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    s->last_stream = stream;
    s->last_launches = 0;
    dresd_status st = run_preprocess(s, queries, B, ((B + 7) / 8) * 8, stream);
    if (st != DRESD_OK) return st;
    cudaError_t e = cudaMemcpyAsync(out_qhat, s->qhat, sizeof(float) * (size_t)B * s->d,
                                    cudaMemcpyDeviceToDevice, stream);
    if (e != cudaSuccess) return fail_cuda(e, "qhat copy");
    return DRESD_OK;
}

dresd_status dresd_store_status(dresd_store *s)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    cudaError_t e = cudaStreamSynchronize(s->last_stream);
    if (e != cudaSuccess) return fail_cuda(e, "stream synchronize");
    int word = 0;
    e = cudaMemcpy(&word, s->status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(e, "status read");
    if (word != 0) {
        cudaMemset(s->status, 0, sizeof(int));
        if (word <= -1000)
            return fail(DRESD_ERR_INTERNAL, "debug build: bounds check %d failed (an index or ring slot out of range)",
                        -1000 - word);
        return fail(DRESD_ERR_TIMEOUT, "a device-side wait expired");
    }
    return DRESD_OK;
}

int dresd_debug_build(void)
{
#ifdef DRESD_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

dresd_status dresd_store_debug_selftest(dresd_store *s, void *stream)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
#ifdef DRESD_DEBUG_BOUNDS
    s->last_stream = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_debug_selftest(s->status, s->last_stream);
    return e == cudaSuccess ? DRESD_OK : fail_cuda(e, "selftest launch");
#else
    (void)stream;
    return fail(DRESD_ERR_UNSUPPORTED, "this is the release build: no bounds checks are compiled in");
#endif
}

dresd_status dresd_store_set_option(dresd_store *s, const char *name, int value)
{
    if (!valid(s) || !name) return fail(DRESD_ERR_INVALID, "store handle or name is NULL");
    if (strcmp(name, "scan_path") == 0) {
        if (value < 0 || value > 2) return fail(DRESD_ERR_INVALID, "scan_path = %d outside 0..2", value);
        s->opt_path = value;
        return DRESD_OK;
    }
    if (strcmp(name, "debug_no_select") == 0) {
        s->opt_no_select = value;
        return DRESD_OK;
    }
    if (strcmp(name, "wait_ms") == 0) {
        if (value < 0 || value > 60000) return fail(DRESD_ERR_INVALID, "wait_ms = %d outside 0..60000", value);
        s->opt_wait_ms = value;
        return DRESD_OK;
    }
    if (strcmp(name, "debug_lose_stage") == 0) {
        if (value < 0) return fail(DRESD_ERR_INVALID, "debug_lose_stage = %d is negative", value);
        s->opt_lose_stage = value;
        return DRESD_OK;
    }
    if (strcmp(name, "pack2") == 0) {
        if (value != 0 && value != 1) return fail(DRESD_ERR_INVALID, "pack2 takes 0 or 1");
        s->opt_pack2 = value;
        return DRESD_OK;
    }
    if (strcmp(name, "first_token_windows") == 0) {
        if (value != 0 && value != 1) return fail(DRESD_ERR_INVALID, "first_token_windows takes 0 or 1");
        s->opt_windows = value;
        return DRESD_OK;
    }
    if (strcmp(name, "merge_level") == 0) {
        if (value < 0 || value > 32) return fail(DRESD_ERR_INVALID, "merge_level outside 0..32");
        s->opt_merge_level = value;
        return DRESD_OK;
    }
    if (strcmp(name, "epi_warps") == 0) {
        if (value != 0 && value != 8 && value != 16) return fail(DRESD_ERR_INVALID, "epi_warps takes 0, 8 or 16");
        s->opt_epi_warps = value;
        return DRESD_OK;
    }
    if (strcmp(name, "fast_reject") == 0) {
        if (value != 0 && value != 1) return fail(DRESD_ERR_INVALID, "fast_reject takes 0 or 1");
        s->opt_no_fast_reject = !value;
        return DRESD_OK;
    }
    if (strcmp(name, "round_per_tile") == 0) {
        if (value != 0 && value != 1) return fail(DRESD_ERR_INVALID, "round_per_tile takes 0 or 1");
        s->opt_round_per_tile = value;
        return DRESD_OK;
    }
    if (strcmp(name, "merged_columns") == 0) {
        if (value < 0 || value > 2) return fail(DRESD_ERR_INVALID, "merged_columns = %d outside 0..2", value);
        s->opt_merged = value;
        return DRESD_OK;
    }
    if (strcmp(name, "keys_as_m") == 0) {
        if (value != 0 && value != 1) return fail(DRESD_ERR_INVALID, "keys_as_m takes 0 or 1");
        s->opt_keys_as_m = value;
        return DRESD_OK;
    }
    if (strcmp(name, "probe") == 0) {
        if (value < 0 || value > 65536) return fail(DRESD_ERR_INVALID, "probe = %d outside 0..65536", value);
        s->opt_probe = value;
        return DRESD_OK;
    }
    if (strcmp(name, "grid") == 0) {
        if (value < 0 || value > s->max_grid) return fail(DRESD_ERR_INVALID, "grid = %d outside 0..%d", value, s->max_grid);
        s->opt_grid = value;
        return DRESD_OK;
    }
    if (strcmp(name, "profile_stride") == 0) {
        if (value < 1 || value > 65536) return fail(DRESD_ERR_INVALID, "profile_stride = %d outside 1..65536", value);
        s->prof_stride = value;
        s->prof_calls = 0;
        return DRESD_OK;
    }
    if (strcmp(name, "profile") == 0) {
        if (value < 0 || value > 65536) return fail(DRESD_ERR_INVALID, "profile = %d outside 0..65536", value);
        for (int i = 0; i < 2 * s->prof_cap; ++i) cudaEventDestroy(s->prof_events[i]);
        delete[] s->prof_events;
        s->prof_events = nullptr;
        s->prof_cap = s->prof_count = 0;
        if (value > 0) {
            s->prof_events = new (std::nothrow) cudaEvent_t[2 * (size_t)value];
            if (!s->prof_events) return fail(DRESD_ERR_ALLOC, "host allocation failed");
            for (int i = 0; i < 2 * value; ++i)
                if (cudaEventCreate(&s->prof_events[i]) != cudaSuccess) {
                    for (int j = 0; j < i; ++j) cudaEventDestroy(s->prof_events[j]);
                    delete[] s->prof_events;
                    s->prof_events = nullptr;
                    return fail(DRESD_ERR_CUDA, "cudaEventCreate failed");
                }
            s->prof_cap = value;
        }
        return DRESD_OK;
    }
    return fail(DRESD_ERR_INVALID, "unknown option '%s'", name);
}

dresd_status dresd_store_profile_read(dresd_store *s, double *scan_ms_total, int *calls)
{
    if (!valid(s) || !scan_ms_total || !calls) return fail(DRESD_ERR_INVALID, "NULL argument");
    cudaError_t e = cudaStreamSynchronize(s->last_stream);
    if (e != cudaSuccess) return fail_cuda(e, "stream synchronize");
    double total = 0.0;
    for (int i = 0; i < s->prof_count; ++i) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, s->prof_events[2 * i], s->prof_events[2 * i + 1]);
        if (e != cudaSuccess) return fail_cuda(e, "cudaEventElapsedTime");
        total += ms;
    }
    *scan_ms_total = total;
    *calls = s->prof_count;
    s->prof_count = 0;
    return DRESD_OK;
}

dresd_status dresd_drafts_prepare(const int32_t *tokens, const int32_t *ids, int B, int n, int L, int32_t eos_id,
                                  int32_t *out_drafts, int32_t *out_valid, void *stream)
{
    if (B < 0 || n < 1 || L < 1) return fail(DRESD_ERR_INVALID, "bad B/n/L");
    if (n > DRESD_MAX_TOP_N) return fail(DRESD_ERR_UNSUPPORTED, "n = %d exceeds DRESD_MAX_TOP_N", n);
    if ((size_t)n * L * sizeof(int32_t) > 48 * 1024) return fail(DRESD_ERR_UNSUPPORTED, "n * L = %d exceeds 12288", n * L);
    if (B == 0) return DRESD_OK;
    if (!is_device_ptr(tokens) || !is_device_ptr(ids) || !is_device_ptr(out_drafts) || !is_device_ptr(out_valid))
        return fail(DRESD_ERR_INVALID, "tokens/ids/out_* must be device pointers");
    cudaError_t e = launch_drafts_prepare(tokens, ids, B, n, L, eos_id, out_drafts, out_valid,
                                          static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? DRESD_OK : fail_cuda(e, "drafts_prepare launch");
}

dresd_status dresd_drafts_accept(const int32_t *drafts, const int32_t *valid, const int32_t *llm_tokens, int B,
                                 int n, int L, int32_t *out_best, int32_t *out_len, int32_t *out_tokens,
                                 void *stream)
{
    if (B < 0 || n < 1 || L < 1) return fail(DRESD_ERR_INVALID, "bad B/n/L");
    if (n > DRESD_MAX_TOP_N) return fail(DRESD_ERR_UNSUPPORTED, "n = %d exceeds DRESD_MAX_TOP_N", n);
    if (B == 0) return DRESD_OK;
    if (!is_device_ptr(drafts) || !is_device_ptr(valid) || !is_device_ptr(llm_tokens) || !is_device_ptr(out_best) ||
        !is_device_ptr(out_len) || !is_device_ptr(out_tokens))
        return fail(DRESD_ERR_INVALID, "all buffers must be device pointers");
    cudaError_t e = launch_drafts_accept(drafts, valid, llm_tokens, B, n, L, out_best, out_len, out_tokens,
                                         static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? DRESD_OK : fail_cuda(e, "drafts_accept launch");
}

dresd_status dresd_merge_shards(const int32_t *ids, const float *scores, const int32_t *tokens,
                                const int64_t *row_offsets, int P, int B, int top_n, int draft_len,
                                int32_t *out_ids, float *out_scores, int32_t *out_tokens, void *stream)
{
    if (P < 1 || B < 0 || top_n < 1 || draft_len < 1) return fail(DRESD_ERR_INVALID, "bad P/B/top_n/draft_len");
    if (top_n > DRESD_MAX_TOP_N) return fail(DRESD_ERR_UNSUPPORTED, "top_n = %d exceeds DRESD_MAX_TOP_N", top_n);
    if (B == 0) return DRESD_OK;
    if (!is_device_ptr(ids) || !is_device_ptr(scores) || !is_device_ptr(tokens) || !is_device_ptr(row_offsets) ||
        !is_device_ptr(out_ids) || !is_device_ptr(out_scores) || !is_device_ptr(out_tokens))
        return fail(DRESD_ERR_INVALID, "all buffers must be device pointers");
    cudaError_t e = launch_merge_shards(ids, scores, tokens, (size_t)B * top_n, (size_t)B * top_n,
                                        (size_t)B * top_n * draft_len, reinterpret_cast<const long long *>(row_offsets), P,
                                        B, top_n, draft_len, out_ids, out_scores, out_tokens,
                                        static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? DRESD_OK : fail_cuda(e, "merge_shards launch");
}

dresd_status dresd_merge_shards_packed(const int32_t *packed, const int64_t *row_offsets, int P, int B, int top_n,
                                       int draft_len, int32_t *out_ids, float *out_scores, int32_t *out_tokens,
                                       void *stream)
{
    if (P < 1 || B < 0 || top_n < 1 || draft_len < 1) return fail(DRESD_ERR_INVALID, "bad P/B/top_n/draft_len");
    if (top_n > DRESD_MAX_TOP_N) return fail(DRESD_ERR_UNSUPPORTED, "top_n = %d exceeds DRESD_MAX_TOP_N", top_n);
    if (B == 0) return DRESD_OK;
    if (!is_device_ptr(packed) || !is_device_ptr(row_offsets) || !is_device_ptr(out_ids) || !is_device_ptr(out_scores) ||
        !is_device_ptr(out_tokens))
        return fail(DRESD_ERR_INVALID, "all buffers must be device pointers");
    const size_t bn = (size_t)B * top_n, block = bn * (2 + (size_t)draft_len);
    cudaError_t e = launch_merge_shards(packed, reinterpret_cast<const float *>(packed + bn), packed + 2 * bn, block, block,
                                        block, reinterpret_cast<const long long *>(row_offsets), P, B, top_n, draft_len,
                                        out_ids, out_scores, out_tokens, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? DRESD_OK : fail_cuda(e, "merge_shards launch");
}

dresd_status dresd_build_keys(const void *hidden, int64_t N, int d_in, dresd_dtype dtype, const float *mean,
                              const float *var, float eps_z, const void *W, int d, const float *pca_mean,
                              void *out_keys, void *stream_v)
{
    if (dtype != DRESD_F16 && dtype != DRESD_BF16)
        return fail(DRESD_ERR_UNSUPPORTED, "dresd_build_keys builds 16-bit datastores (fp16 or bf16)");
    if (N <= 0 || N > kMaxRows) return fail(DRESD_ERR_INVALID, "N = %lld outside 1..2^31-1024", (long long)N);
    if (d_in < 8 || d_in % 8 != 0) return fail(DRESD_ERR_INVALID, "d_in = %d must be a positive multiple of 8", d_in);
    if (d < 32 || d > 256 || d % 32 != 0) return fail(DRESD_ERR_UNSUPPORTED, "d = %d must be 32..256 in steps of 32", d);
    if (d_in > 16384) return fail(DRESD_ERR_UNSUPPORTED, "d_in = %d exceeds 16384", d_in);
    if ((mean == nullptr) != (var == nullptr)) return fail(DRESD_ERR_INVALID, "mean and var go together");
    if (!(eps_z >= 0.f)) return fail(DRESD_ERR_INVALID, "eps_z must be >= 0");
    if (!is_device_ptr(hidden) || !is_device_ptr(W) || !is_device_ptr(out_keys) || (mean && !is_device_ptr(mean)) ||
        (var && !is_device_ptr(var)) || (pca_mean && !is_device_ptr(pca_mean)))
        return fail(DRESD_ERR_INVALID, "hidden/W/out_keys/mean/var/pca_mean must be device pointers");
    if (reinterpret_cast<uintptr_t>(hidden) % 16 != 0 || reinterpret_cast<uintptr_t>(out_keys) % 16 != 0)
        return fail(DRESD_ERR_INVALID, "hidden / out_keys not 16-byte aligned");
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDevice");
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return fail_cuda(e, "SM count");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);

    const size_t kpad = ((size_t)d_in + 63) / 64 * 64;
    if (dev < 0 || dev >= kScratchDevices) return fail(DRESD_ERR_UNSUPPORTED, "device ordinal beyond 63");
    std::lock_guard<std::mutex> ws_lock(g_scratch_mutex);      // one build per device at a time
    uint8_t *ws = device_scratch(dev, build_keys_workspace_bytes(d_in, d));
    if (!ws) return fail(DRESD_ERR_ALLOC, "workspace allocation failed");
    void *wt_hi = ws, *wt_lo = ws + (size_t)d * kpad * 2;
    float *bias = reinterpret_cast<float *>(ws + 2 * (size_t)d * kpad * 2);
    int *status = reinterpret_cast<int *>(bias + 256);
    dresd_status st = DRESD_OK;
    CUtensorMap h_map, whi_map, wlo_map;
    const int pair = g_build_pairs.load() != 0 ? 1 : 0;            // CTA pairs stage half of W' each
    const int w_box = pair ? d / 2 : d;
    if (!make_map(&h_map, hidden, (int)dtype, N, d_in, 128) ||
        !make_map(&whi_map, wt_hi, (int)dtype, d, (int)kpad, w_box) ||
        !make_map(&wlo_map, wt_lo, (int)dtype, d, (int)kpad, w_box))
        st = fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled failed");
    if (st == DRESD_OK && (e = cudaMemsetAsync(status, 0, sizeof(int), stream)) != cudaSuccess)
        st = fail_cuda(e, "status reset");
    if (st == DRESD_OK && (e = launch_build_prep(W, (int)dtype, mean, var, eps_z, pca_mean, d_in, d, wt_hi, wt_lo, bias,
                                                 stream)) != cudaSuccess)
        st = fail_cuda(e, "build prep launch");
    if (st == DRESD_OK && (e = launch_build_keys(h_map, whi_map, wlo_map, (int)dtype, N, d_in, d, mean ? 2 : 1, pair, bias, out_keys,
                                                 kEpsNorm, status, sms, stream, (long long)g_build_wait_ms.load() * 2000000LL,
                                                 g_build_lose_stage.load())) != cudaSuccess)
        st = fail_cuda(e, "build keys launch");
    int word = 0;
    if (st == DRESD_OK && (e = cudaMemcpyAsync(&word, status, sizeof(int), cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        st = fail_cuda(e, "status read");
    e = cudaStreamSynchronize(stream);                 // the scratch is reused by the next call
    if (st == DRESD_OK && e != cudaSuccess) st = fail_cuda(e, "stream synchronize");
    if (st == DRESD_OK && word != 0) st = fail(DRESD_ERR_TIMEOUT, "a device-side wait expired");
    return st;
}

dresd_status dresd_quantise_keys(const void *keys, int64_t N, int d, dresd_dtype dtype, void *out_q8, void *stream)
{
    if (dtype != DRESD_F16 && dtype != DRESD_BF16)
        return fail(DRESD_ERR_UNSUPPORTED, "dresd_quantise_keys reads 16-bit datastores (fp16 or bf16)");
    if (N <= 0 || N > kMaxRows) return fail(DRESD_ERR_INVALID, "N = %lld outside 1..2^31-1024", (long long)N);
    if (d < 16 || d % 16 != 0) return fail(DRESD_ERR_INVALID, "d = %d must be a positive multiple of 16", d);
    if (!is_device_ptr(keys) || !is_device_ptr(out_q8)) return fail(DRESD_ERR_INVALID, "keys / out_q8 must be device pointers");
    if (reinterpret_cast<uintptr_t>(keys) % 16 != 0 || reinterpret_cast<uintptr_t>(out_q8) % 16 != 0)
        return fail(DRESD_ERR_INVALID, "keys / out_q8 not 16-byte aligned");
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return fail_cuda(e, "device query");
    e = launch_quantise_keys(keys, (int)dtype, N, d, out_q8, sms, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? DRESD_OK : fail_cuda(e, "quantise launch");
}

dresd_status dresd_store_attach_quantised(dresd_store *s, const void *keys_q8)
{
    if (!valid(s)) return fail(DRESD_ERR_INVALID, "store handle is NULL or destroyed");
    if (s->dtype == kF32) return fail(DRESD_ERR_UNSUPPORTED, "the quantised search needs a 16-bit store");
    if (s->d % 16 != 0) return fail(DRESD_ERR_UNSUPPORTED, "d = %d must be a multiple of 16 for the 8-bit copy", s->d);
    if (s->d > 2048) return fail(DRESD_ERR_UNSUPPORTED, "d = %d exceeds 2048 for the 8-bit copy", s->d);
    if (!is_device_ptr(keys_q8) || reinterpret_cast<uintptr_t>(keys_q8) % 16 != 0)
        return fail(DRESD_ERR_INVALID, "keys_q8 must be a 16-byte aligned device pointer");
    s->k8 = nullptr;                  // a failed attach leaves no copy attached
    if (!s->qsplit8) {
        s->dpad8 = (s->d + 127) / 128 * 128;
        if (cudaMalloc(&s->qsplit8, (size_t)2 * kMaxBatch * s->dpad8) != cudaSuccess) {
            cudaGetLastError();
            s->qsplit8 = nullptr;
            return fail(DRESD_ERR_ALLOC, "workspace allocation failed");
        }
    }
    // The scan kernels see the 8-bit store as rows of d/2 two-byte units (TMA moves bytes).
    bool ok = make_map(&s->map_k8, keys_q8, kF16, s->N, s->d / 2, 128);
    for (int i = 0; i < 4; ++i) ok = ok && make_map(&s->map_q8[i], s->qsplit8, kF16, 2 * kMaxBatch, s->dpad8 / 2, 16 << i);
    if (!ok) return fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the 8-bit copy");
    s->k8_packable = 0;
    if (s->d == 64 && s->N >= 2) {
        if (!make_map(&s->map_k8p, keys_q8, kF16, s->N / 2, 64, 128))
            return fail(DRESD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the packed 8-bit copy");
        s->k8_packable = 1;
    }
    s->k8 = keys_q8;
    return DRESD_OK;
}

dresd_status dresd_retrieve_quantised(dresd_store *s, const void *queries, const int32_t *first_tokens, int B,
                                      int top_n, int draft_len, int candidates, int32_t *out_ids, float *out_scores,
                                      int32_t *out_tokens, void *stream)
{
    dresd_status st = check_retrieve_args(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens, true);
    if (st != DRESD_OK) return st;
    if (first_tokens) {
        if (!s->first_col) return fail(DRESD_ERR_INVALID, "call dresd_store_enable_first_token_filter() first");
        if (B > 0 && !is_device_ptr(first_tokens)) return fail(DRESD_ERR_INVALID, "first_tokens must be a device pointer");
    }
    if (!s->k8) return fail(DRESD_ERR_INVALID, "no 8-bit copy attached (dresd_store_attach_quantised)");
    if (candidates < top_n || candidates > DRESD_MAX_TOP_N || candidates > s->N)
        return fail(DRESD_ERR_INVALID, "candidates = %d outside top_n..min(%d, N)", candidates, DRESD_MAX_TOP_N);
    if (B == 0) return DRESD_OK;
    return run_retrieve(s, queries, B, top_n, draft_len, out_ids, out_scores, out_tokens,
                        static_cast<cudaStream_t>(stream), first_tokens, candidates);
}

dresd_status dresd_set_global_option(const char *name, int value)
{
    if (!name) return fail(DRESD_ERR_INVALID, "option name is NULL");
    if (std::strcmp(name, "build_keys_pairs") == 0) {
        if (value != 0 && value != 1) return fail(DRESD_ERR_INVALID, "build_keys_pairs takes 0 or 1");
        g_build_pairs.store(value);
        return DRESD_OK;
    }
    if (std::strcmp(name, "build_keys_wait_ms") == 0) {
        if (value < 0 || value > 60000) return fail(DRESD_ERR_INVALID, "build_keys_wait_ms = %d outside 0..60000", value);
        g_build_wait_ms.store(value);
        return DRESD_OK;
    }
    if (std::strcmp(name, "build_keys_debug_lose_stage") == 0) {
        if (value < 0) return fail(DRESD_ERR_INVALID, "build_keys_debug_lose_stage = %d is negative", value);
        g_build_lose_stage.store(value);
        return DRESD_OK;
    }
    return fail(DRESD_ERR_INVALID, "unknown global option '%s'", name);
}

dresd_status dresd_fit_zscore(const void *sample, int64_t N, int d_in, dresd_dtype dtype, float *out_mean,
                              float *out_var, void *stream_v)
{
    if (dtype != DRESD_F16 && dtype != DRESD_BF16)
        return fail(DRESD_ERR_UNSUPPORTED, "dresd_fit_zscore reads 16-bit embeddings (fp16 or bf16)");
    if (N <= 0) return fail(DRESD_ERR_INVALID, "N = %lld must be positive", (long long)N);
    if (d_in < 8 || d_in % 8 != 0) return fail(DRESD_ERR_INVALID, "d_in = %d must be a positive multiple of 8", d_in);
    if (d_in > 16384) return fail(DRESD_ERR_UNSUPPORTED, "d_in = %d exceeds 16384", d_in);
    if (!is_device_ptr(sample) || !is_device_ptr(out_mean) || !is_device_ptr(out_var))
        return fail(DRESD_ERR_INVALID, "sample/out_mean/out_var must be device pointers");
    if (reinterpret_cast<uintptr_t>(sample) % 16 != 0) return fail(DRESD_ERR_INVALID, "sample not 16-byte aligned");
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDevice");
    if (dev < 0 || dev >= kScratchDevices) return fail(DRESD_ERR_UNSUPPORTED, "device ordinal beyond 63");
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return fail_cuda(e, "SM count");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    std::lock_guard<std::mutex> ws_lock(g_scratch_mutex);
    uint8_t *ws = device_scratch(dev, fit_zscore_workspace_bytes(N, d_in, sms));
    if (!ws) return fail(DRESD_ERR_ALLOC, "workspace allocation failed");
    dresd_status st = DRESD_OK;
    if ((e = launch_fit_zscore(sample, (int)dtype, N, d_in, sms, ws, out_mean, out_var, stream)) != cudaSuccess)
        st = fail_cuda(e, "fit_zscore launch");
    e = cudaStreamSynchronize(stream);                 // the scratch is reused by the next call
    if (st == DRESD_OK && e != cudaSuccess) st = fail_cuda(e, "stream synchronize");
    return st;
}

int dresd_store_last_launches(const dresd_store *s) { return valid(s) ? s->last_launches : 0; }

double dresd_store_last_key_passes(const dresd_store *s) { return valid(s) ? s->last_key_passes : 0.0; }

const char *dresd_last_error(void) { return g_err; }

void dresd_store_destroy(dresd_store *s)
{
    if (valid(s)) free_store(s);
}

}  // extern "C"

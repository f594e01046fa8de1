// Host-side declarations shared by the kernel files and the C ABI (api.cu).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dresd {

enum { kF32 = 0, kF16 = 1, kBF16 = 2, kE4M3 = 3 };   // kE4M3: the 8-bit copy of a 16-bit store (internal)

constexpr int kMaxBatch = 64;
constexpr int kMaxTopN = 32;
constexpr int kCandStride = 32;          // u64 slots per (CTA, query) in the workspace
constexpr long long kMaxRows = 2147483647LL - 1023;   // row coordinates of the last (partly filled) tile stay within int32
constexpr float kHiLoScaleF16 = 2048.f;  // low half of an fp16-split query is stored x 2^11
constexpr float kHiLoScaleBF16 = 256.f;  // low half of a bf16-split query is stored x 2^8

// ---- K1: Eq. 1 -> v W -> Eq. 2 -------------------------------------------
struct PreprocessArgs {
    const void *queries;    // [B][d_in] store dtype
    const float *mean;      // [d_in] or null
    const float *var;       // [d_in] or null
    const void *W;          // [d_in][d] store dtype or null
    const float *pca_mean;  // [d_in] or null
    float eps_z, eps_n;
    int B, d_in, d, dtype;
    float *qhat;            // [rows][d] fp32 unit queries (rows >= B zero)
    void *qsplit;           // 16-bit keys: [2*rows][dpad] hi/lo operand rows, else null
    int dpad;               // d rounded up to 64
    int rows;               // CTAs launched: B rounded up to the operand row count
    float lo_scale;
    unsigned int *gtau;     // [rows] grid-wide filter words, reset to 0 ("nothing known") here
    int split_blocked;      // qsplit rows: 0 = (2b, 2b+1); 1 = 16-row blocks, hi rows 0-7, lo rows 8-15;
                            // 2 = rows b and `rows` + b hold S hi and S (q - hi), S = lo_scale (one column per query);
                            // 4 = rows b and `rows` + b hold hi and S (q - hi): two columns per query, hi columns first;
                            // 3 = d = 32 keys scanned two per 64-element row: rows 4b .. 4b+3 = (hi|0), (lo|0), (0|hi), (0|lo)
    // Split projection (W given): `slices` CTAs of `rows_per_slice` rows of W each write
    // partial[slice][B][d]; null = every query's CTA walks all of W itself.
    float *partial;
    int slices, rows_per_slice;
    // Quantised search: also write the two E4M3 terms of every query (see store_query_e4m3); null = not needed.
    uint8_t *qsplit8;
    int dpad8, pack2;
};
// Slices and rows per slice of the split projection for a workspace of `bytes` (0 slices = do not split).
void preprocess_split_plan(int d_in, int d, int B, int elem_bytes, size_t bytes, int *slices, int *rows_per_slice);
cudaError_t launch_preprocess(const PreprocessArgs &a, cudaStream_t stream);

// ---- K2+K3: score every key, keep a per-CTA top-n per query ----------------
struct ScanArgs {
    long long N;            // rows
    int d;                  // key dimension
    int dpad;               // row length of qsplit (multiple of 64)
    int dtype;
    int n_tiles;            // row tiles of the kernel's tile height
    int B;                  // queries handled by this launch
    int top_n;
    const float *qhat;      // fp32 unit queries of this launch, [B][d]
    const void *qsplit;     // hi/lo operand rows of this launch, [2*Bpad][dpad]
    float lo_inv_scale;     // 1 / lo_scale
    unsigned long long *cand;  // [grid][cand_batch][kCandStride], at this launch's first query
    int cand_batch;         // query stride of `cand` (the call's B)
    int *status;            // device status word
    unsigned int *gtau;     // grid-wide filter words of this launch's queries (see share_tau)
    // First-token filter (Section 3.5): when both are set, query q only accepts rows
    // with first_col[row] == want_first[q]; want_first[q] < 0 disables it for that query.
    const int32_t *first_col;   // [N] first stored token of every key (compact copy)
    const int32_t *want_first;  // [B] of this launch
    // Store sorted by first token (tcgen05 kernel with the keys as M): win_start[t] .. win_start[t+1]
    // are the rows whose first token is t, t < win_vocab.  When every query of the launch names a
    // token, only those windows are scanned; the result is that of the filtered full scan.
    const int32_t *win_start;   // [win_vocab + 1], null = always scan everything
    int win_vocab;
    int stages;             // pipeline depth
    long long wait_cycles;  // bound of every device-side wait in cycles, 0 = default (~2 s)
    int debug_lose_stage;   // test hook (every scan kernel): CTA 0 never receives stage (value-1); 0 = off
    int tile_stride;        // tcgen05 kernel: visit every tile_stride-th tile (probe pass), default 1
    int probe_max;          // tcgen05 kernel, probe pass: keep only each tile's best row per query
    int no_select;          // tcgen05 kernel, measurement only: nothing passes the filter (scan floor)
    int keys_as_m;          // tcgen05 kernels: never use the form with the keys as the N = 256 operand
    int merge_level;        // tcgen05 kernels: a round is asked for when a queue holds this many (0 = 16) (measurement)
    int epi_warps;          // tcgen05 kernel, one column per query: 16 = sixteen epilogue warps (measurement)
    int no_fast_reject;     // tcgen05 kernel, keys as N: skip the packed sign-bit rejection ahead of the exact compare (measurement)
    int round_per_tile;     // tcgen05 kernel, keys as M: the epilogue warps meet at every tile (measurement)
    int merged;             // tcgen05 kernel, keys as M: one accumulator column per query (operand: hi' rows, then lo' rows)
    int pack2;              // 64-byte keys (8-bit d = 64, 16-bit d = 32): a 128-byte row holds two keys (N = rows, ids = 2 row + parity)
};
// Tile heights (rows per TMA stage) so that api.cu can build matching tensor maps.
int scan_mma_tile_rows(int d);
int scan_mma_queries_per_launch(int d, int B);
size_t scan_mma_smem_bytes(int d, int B, int *stages_out);
cudaError_t launch_scan_mma(const CUtensorMap &keys_map, const ScanArgs &a, int grid,
                            cudaStream_t stream);

// Batched tensor-core kernel (tcgen05/TMEM, 16-bit keys): 128-row tiles; the query
// operand holds 2 rows per query, padded to 16/32/64/128 rows.
int scan_umma_tile_rows(int d, int B, int keys_as_m, int merged);   // rows per tile of the kernel that will run
bool scan_umma_merged_eligible(int d, int B, int dtype);            // one accumulator column per query
// 16-bit keys of 32 elements scanned as rows of two keys (the packed forms of the kernel for 16-bit operands)
cudaError_t launch_scan_umma_pack16(const CUtensorMap &keys_map, const CUtensorMap &q_map, const ScanArgs &a,
                                    int grid, cudaStream_t stream);
cudaError_t launch_scan_umma_merged(const CUtensorMap &keys_map, const CUtensorMap &q_map, const ScanArgs &a,
                                    int grid, cudaStream_t stream);
int scan_umma_operand_rows(int B);
cudaError_t launch_scan_umma(const CUtensorMap &keys_map, const CUtensorMap &q_map, const ScanArgs &a,
                             int grid, cudaStream_t stream);

// Same path for 17-64 queries on rows of 129-256 elements: queries as the M = 128 operand,
// keys as the N = 256 operand (256-key tiles).  launch_scan_umma() dispatches to it.
bool scan_ummat_eligible(int d, int B);
cudaError_t launch_scan_ummat(const CUtensorMap &keys_map, const CUtensorMap &q_map, const ScanArgs &a,
                              int grid, cudaStream_t stream);

int scan_f32_tile_rows(int d);   // rows per tile (tile count)
int scan_f32_box_rows(int d);    // rows per TMA box of the key map (a tile is fetched as several boxes)
int scan_f32_queries_per_launch(int d, int B);
cudaError_t launch_scan_f32(const CUtensorMap &keys_map, const ScanArgs &a, int grid,
                            cudaStream_t stream);

// ---- K4: merge the per-CTA lists;  K5: gather continuations ----------------
// Merge of the per-CTA lists and gather of the winners' stored tokens, one kernel.
cudaError_t launch_merge_gather(const unsigned long long *cand, int grid_lists, int B, int top_n, int32_t *out_ids,
                                float *out_scores, const int32_t *next_tokens, int stored_len, long long N,
                                int draft_len, int32_t *out_tokens, cudaStream_t stream, int *status = nullptr);
// Same merge, but only the n-th best score of each query is kept, as a grid-wide
// filter word (see share_tau); 0 when fewer than top_n candidates exist.
cudaError_t launch_merge_tau(const unsigned long long *cand, int grid_lists, int B, int top_n,
                             unsigned int *gtau, cudaStream_t stream);

// first_col[i] = next_tokens[i][0]: the compact column the first-token filter reads.
cudaError_t launch_extract_first(const int32_t *next_tokens, int stored_len, long long N,
                                 int32_t *first_col, cudaStream_t stream);

// Index of a store whose rows are sorted by first token.  check: *flag gets bit 0 when
// first_col is not non-decreasing, bit 1 when it holds a negative token.  build:
// win_start[t] = first row with first token >= t for t = 0 .. vocab (vocab = last token + 1).
cudaError_t launch_check_sorted(const int32_t *first_col, long long N, int *flag, cudaStream_t stream);
cudaError_t launch_build_windows(const int32_t *first_col, long long N, int vocab, int32_t *win_start,
                                 cudaStream_t stream);

// ---- K6: draft matrix preparation and longest-match acceptance (Section 3.6) ----
cudaError_t launch_drafts_prepare(const int32_t *tokens, const int32_t *ids, int B, int n, int L, int eos,
                                  int32_t *drafts, int32_t *valid, cudaStream_t stream);
cudaError_t launch_drafts_accept(const int32_t *drafts, const int32_t *valid, const int32_t *llm, int B, int n,
                                 int L, int32_t *out_best, int32_t *out_len, int32_t *out_tokens,
                                 cudaStream_t stream);

// Exchange step of a row-sharded datastore: P per-shard top-n lists -> the global top-n.
cudaError_t launch_merge_shards(const int32_t *ids, const float *scores, const int32_t *tokens, size_t stride_ids,
                                size_t stride_scores, size_t stride_tokens, const long long *offsets, int P, int B,
                                int n, int L, int32_t *out_ids, float *out_scores, int32_t *out_tokens,
                                cudaStream_t stream);

// ---- K7: datastore-side preprocessing (Eq. 1 -> v W -> Eq. 2 over N rows), a tcgen05 GEMM ----
// `terms` = 2 multiplies by W' = hi + lo (needed when Eq. 1 scales the weights), 1 by hi alone
// (exact when there is no z-score: W' is W).  `pair` != 0 runs the kernel on CTA pairs
// (cta_group::2, clusters of two); the W' tensor maps must then have boxes of d/2 rows.
size_t build_keys_workspace_bytes(int d_in, int d);
cudaError_t launch_build_prep(const void *W, int dtype, const float *mean, const float *var, float eps_z,
                              const float *pca_mean, int d_in, int d, void *wt_hi, void *wt_lo, float *bias,
                              cudaStream_t stream);
cudaError_t launch_build_keys(const CUtensorMap &h_map, const CUtensorMap &whi_map, const CUtensorMap &wlo_map,
                              int dtype, long long N, int d_in, int d, int terms, int pair, const float *bias,
                              void *out, float eps_n, int *status, int grid, cudaStream_t stream,
                              long long wait_cycles = 0, int lose_stage = 0);

// ---- K8: statistics of Eq. 1 (Section 3.2) from a sample of embeddings, one streaming pass ----
size_t fit_zscore_workspace_bytes(long long N, int d_in, int sms);
cudaError_t launch_fit_zscore(const void *V, int dtype, long long N, int d_in, int sms, void *workspace,
                              float *mean, float *var, cudaStream_t stream);

// ---- K9: quantised candidate search (8-bit E4M3 keys, exact re-ranking) ----
cudaError_t launch_quantise_keys(const void *keys, int dtype, long long N, int d, void *out_q8, int sms,
                                 cudaStream_t stream);
// Fold of the per-CTA approximate lists, exact re-ranking of the survivors, value lookup: one kernel.
// extra_id >= 0: one more candidate for every query (the last key of an odd-sized packed store).
cudaError_t launch_merge_rerank(const unsigned long long *cand, int lists, int B, const void *keys, int dtype, int d,
                                long long N, const float *qhat, int mcand, int top_n, long long extra_id,
                                const int32_t *want_first, const int32_t *next_tokens, int stored_len, int draft_len,
                                int32_t *out_ids, float *out_scores, int32_t *out_tokens, cudaStream_t stream);

// Debug build only: one thread fails check 7 on purpose (no access is attempted), to show the reporting path.
cudaError_t launch_debug_selftest(int *status, cudaStream_t stream);

// Stores `msg` as the calling thread's dresd_last_error() text.
void set_last_error(const char *msg);

}  // namespace dresd

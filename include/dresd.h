/*
 * dresd.h -- C ABI of the B200 dense-retrieval draft model of DReSD.
 *
 * One call of dresd_retrieve() is steps 4-7 of the paper's Algorithm 1 for a
 * batch of B decode positions: the query (the LLM's hidden state) is z-scored
 * (Eq. 1), projected to the datastore dimension (Section 3.3, v_l <- v W_l),
 * scaled to unit length (Eq. 2), scored by inner product against EVERY key of
 * the datastore (Eq. 3: cosine similarity, which on unit-length vectors is the
 * inner product; search is exact, not approximate), the top_n best keys are
 * selected, and each one's stored continuation -- the value of the key-value
 * store f_D of Section 3.5 -- is gathered into the n x L draft matrix that
 * batch verification (Section 3.6) consumes.
 *
 * All work runs in CUDA kernels compiled for sm_100a; there is no CPU path.
 * Pointers are DEVICE pointers unless a parameter says "host".  Every function
 * returns a dresd_status (never throws, aborts or exits); when validation
 * fails nothing is enqueued.  dresd_last_error() gives a thread-local message
 * for the last failing call.
 */
#ifndef DRESD_H
#define DRESD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dresd_store dresd_store; /* opaque handle */

typedef enum { DRESD_F32 = 0, DRESD_F16 = 1, DRESD_BF16 = 2 } dresd_dtype;

typedef enum {
    DRESD_OK = 0,
    DRESD_ERR_INVALID = -1,     /* bad pointer / shape / range                        */
    DRESD_ERR_UNSUPPORTED = -2, /* valid request outside the built kernel range       */
    DRESD_ERR_ALLOC = -3,       /* workspace allocation failed                        */
    DRESD_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed                  */
    DRESD_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (see _status)   */
    DRESD_ERR_INTERNAL = -6     /* debug build: a bounds check inside a kernel failed */
} dresd_status;

enum {
    DRESD_MAX_BATCH = 64,  /* largest B per call                                      */
    DRESD_MAX_TOP_N = 32,  /* largest top_n                                           */
    DRESD_MAX_DIM = 4096   /* largest key dimension d                                */
};

/*
 * Section 3.5: the datastore is a key-value store; key = (reduced, unit-length)
 * token embedding, value = the next tokens at that position.
 *
 *   keys         device, [N][d] row-major in `dtype`; base 16-byte aligned and
 *                d * sizeof(dtype) a multiple of 16 (rows are fetched by TMA).
 *   next_tokens  device, int32 [N][stored_len] row-major.
 *   N            1 .. 2^31-1024 rows (tile coordinates are 32-bit);  d: 8 .. DRESD_MAX_DIM.
 *   stored_len   tokens stored per key (the paper's "next N tokens"), >= 1.
 *   out_store    host pointer receiving the handle.
 *
 * Both arrays are BORROWED (zero copy): the caller keeps them alive and
 * unmodified until dresd_store_destroy().  The call allocates a workspace of
 * a few MB on the current device, builds the TMA descriptors and returns; it
 * launches nothing.  A store is bound to the device that was current here and
 * may be used from one stream at a time.
 */
dresd_status dresd_store_create(const void *keys, const int32_t *next_tokens, int64_t N, int d,
                                dresd_dtype dtype, int stored_len, dresd_store **out_store);

/*
 * Optional query preprocessing ahead of the unit-length scaling, Algorithm 1
 * steps 4-5.  Any pointer may be NULL to skip that stage; all are device
 * pointers, borrowed like the keys.
 *
 *   d_in       width of the incoming queries (the LLM hidden size).
 *   mean, var  fp32 [d_in]: E[V] and Var[V] of Eq. 1 (both or neither).
 *   eps_z      the epsilon of Eq. 1 (the paper leaves it open; 1e-5 is usual).
 *   W          [d_in][d] row-major in the store dtype: the first d principal
 *              components, v_l = v W (Section 3.3).  Without W, d_in must be d.
 *   pca_mean   fp32 [d_in] subtracted before the projection, or NULL (the
 *              paper's formula has no centring).
 *
 * Without this call queries are [B][d] and only Eq. 2 is applied.  A set-up call:
 * it may allocate (a staging buffer for the host-buffer call and, with W, 8 MB for
 * the partial products of the projection, which is split over d_in so that W is
 * read once per call for all queries); the retrieval calls allocate nothing.
 */
dresd_status dresd_store_set_preprocess(dresd_store *store, int d_in, const float *mean,
                                        const float *var, float eps_z, const void *W,
                                        const float *pca_mean);

/*
 * Algorithm 1 steps 4-7 for B queries (Eq. 1, Section 3.3, Eq. 2, Eq. 3,
 * Section 3.5), asynchronous on `stream` (a cudaStream_t; NULL = legacy
 * default stream).  No host synchronisation, no allocation.
 *
 *   queries     device, [B][d_in] row-major, same dtype as the keys.
 *   B           0 .. DRESD_MAX_BATCH (0 is a no-op returning DRESD_OK).
 *   top_n       1 .. min(N, DRESD_MAX_TOP_N) neighbours per query.
 *   draft_len   1 .. stored_len tokens copied per neighbour.
 *   out_ids     device, int32 [B][top_n]: row indices, best first; equal
 *               scores are ordered by ascending row index.
 *   out_scores  device, fp32 [B][top_n]: inner product of the unit query with
 *               the stored key (fp32 accumulation).
 *   out_tokens  device, int32 [B][top_n][draft_len]: the first draft_len
 *               stored tokens of each neighbour, verbatim.
 *
 * Non-finite inputs give unspecified results but neither hang nor fault.
 * The call only enqueues kernels: it can be captured into a CUDA graph and replayed
 * (the replay reads the query buffer as it is then; tested).
 */
dresd_status dresd_retrieve(dresd_store *store, const void *queries, int B, int top_n,
                            int draft_len, int32_t *out_ids, float *out_scores,
                            int32_t *out_tokens, void *stream);

/*
 * First-token filter, Sections 3.1 and 3.5: the LLM's own next token x_{t+1}
 * rules out every draft that does not start with it.  The filter is applied
 * BEFORE the selection: query b only considers keys whose first stored token
 * equals first_tokens[b], and returns the top_n best of those.
 *
 * dresd_store_enable_first_token_filter() builds, once per store, a compact
 * int32 [N] copy of next_tokens[.][0] (4 N bytes of device memory, one kernel on
 * `stream`); the scoring kernels read it beside the keys (+4 bytes per row).
 *
 * dresd_retrieve_filtered() is dresd_retrieve() with
 *   first_tokens  device, int32 [B]; a negative entry disables the filter for
 *                 that query; NULL disables it for the call.
 * When fewer than top_n keys match, the missing neighbours are reported as
 * id -1, score -infinity, tokens -1.
 *
 * dresd_store_index_first_tokens() is for a datastore whose rows the caller has
 * SORTED by first stored token (non-decreasing next_tokens[.][0]; row order
 * carries no other meaning, ids are row indices).  It enables the filter if
 * needed, checks the order on the device and builds a table of every token's
 * row range (4 bytes x (largest first token + 2)); it synchronises `stream`.
 * Afterwards a filtered call of the tensor-core path on 16-bit stores (exact or
 * quantised) in which EVERY query names a token scans only those tokens' rows --
 * the result is the one the full filtered scan gives, bit for bit, at a fraction
 * of the bytes; a call with a negative entry in first_tokens scans everything as
 * before.  Returns DRESD_ERR_INVALID when the rows are not sorted or a stored
 * first token is negative, DRESD_ERR_UNSUPPORTED for first tokens >= 2^24.
 * Store option "first_token_windows" = 0 switches the windows off again.
 */
dresd_status dresd_store_enable_first_token_filter(dresd_store *store, void *stream);
dresd_status dresd_store_index_first_tokens(dresd_store *store, void *stream);
dresd_status dresd_retrieve_filtered(dresd_store *store, const void *queries, const int32_t *first_tokens,
                                     int B, int top_n, int draft_len, int32_t *out_ids, float *out_scores,
                                     int32_t *out_tokens, void *stream);

/*
 * Token-level half of batch verification, Section 3.6 and Fig. 3 (no LLM involved).
 *
 * dresd_drafts_prepare() turns the gathered continuations into the n x L draft
 * matrix that is sent for verification:
 *   tokens      device, int32 [B][n][L]  (out_tokens of dresd_retrieve, draft_len = L)
 *   ids         device, int32 [B][n]     (out_ids; -1 = missing neighbour)
 *   out_drafts  device, int32 [B][n][L]: every token after a draft's first eos_id is
 *               eos_id (the EOS id is the padding); a missing neighbour is all eos_id
 *   out_valid   device, int32 [B][n]: 0 for a missing neighbour and for a draft equal
 *               (after padding) to a better-ranked draft of the same query, else 1.
 *
 * dresd_drafts_accept() accepts the longest draft that exactly matches the LLM:
 *   llm_tokens  device, int32 [B][n][L+1]: llm_tokens[b][r][t] is the LLM's own token
 *               at the position of drafts[b][r][t] given the context and the draft's
 *               first t tokens (t = L: the token after the whole draft)
 *   out_best    device, int32 [B]: the valid draft with the longest matching prefix
 *               (ties to the better-ranked one), -1 when no draft is valid
 *   out_len     device, int32 [B]: accepted tokens = matched prefix length + 1
 *   out_tokens  device, int32 [B][L+1]: the matched prefix, then the LLM's token at
 *               the first mismatch (so every step yields at least one token,
 *               Section 3.1), then -1.
 * n <= DRESD_MAX_TOP_N; n * L <= 12288.  Asynchronous on `stream`.
 */
dresd_status dresd_drafts_prepare(const int32_t *tokens, const int32_t *ids, int B, int n, int L,
                                  int32_t eos_id, int32_t *out_drafts, int32_t *out_valid, void *stream);
dresd_status dresd_drafts_accept(const int32_t *drafts, const int32_t *valid, const int32_t *llm_tokens,
                                 int B, int n, int L, int32_t *out_best, int32_t *out_len,
                                 int32_t *out_tokens, void *stream);

/*
 * Datastore-side preprocessing, Sections 3.2-3.5: the KEYS of the datastore are the
 * token embeddings of the corpus after the same three steps the query takes -- Eq. 1
 * (z-scoring), v_l <- v W_l, Eq. 2 (unit length).  This call applies them to N rows of
 * LLM hidden states at once (a tensor-core GEMM [N x d_in] . [d_in x d] with the
 * normalisations fused) and writes the key matrix that dresd_store_create() takes.
 *
 *   hidden     device, [N][d_in] row-major, fp16 or bf16 (`dtype`), 16-byte aligned;
 *              d_in a multiple of 8, at most 16384
 *   mean, var  device fp32 [d_in] (both or neither), eps_z: Eq. 1
 *   W          device, [d_in][d] row-major in `dtype`; d = 32 .. 256 in steps of 32
 *   pca_mean   device fp32 [d_in] or NULL, subtracted after Eq. 1
 *   out_keys   device, [N][d] row-major in `dtype`: unit-length rows, rounded to
 *              `dtype` from fp32 accumulation (hidden states enter exactly; W / sigma
 *              is carried as a two-term 16-bit split; without mean/var W itself is
 *              exact and a single term is multiplied, at half the tensor work)
 *
 * Offline operation: keeps a scratch copy of W per device (4 d d_in bytes, allocated on
 * the first call and reused), runs on `stream` and RETURNS AFTER THE STREAM HAS
 * FINISHED; one build per device at a time.
 */
dresd_status dresd_build_keys(const void *hidden, int64_t N, int d_in, dresd_dtype dtype, const float *mean,
                              const float *var, float eps_z, const void *W, int d, const float *pca_mean,
                              void *out_keys, void *stream);

/*
 * The statistics of Eq. 1, Section 3.2: E[V] and Var[V] per embedding dimension,
 * estimated from a sample V of full-size token embeddings (the paper samples about
 * a million rows of the datastore's hidden states).  Var is the population variance
 * (divide by N; the equation has the batch-normalisation form).  One streaming pass.
 *
 *   sample     device, [N][d_in] row-major, fp16 or bf16 (`dtype`), 16-byte aligned;
 *              N >= 1, d_in a multiple of 8, at most 16384
 *   out_mean   device fp32 [d_in]
 *   out_var    device fp32 [d_in]; exactly 0 for a constant column
 *
 * The outputs are what dresd_store_set_preprocess() and dresd_build_keys() take as
 * mean / var.  Sums are shifted per column and carried in float64, so the result is
 * accurate to fp32 rounding also when |E| >> sqrt(Var); it does not depend on the
 * launch (fixed summation order).  Offline operation like dresd_build_keys(): uses the
 * same per-device scratch, runs on `stream` and RETURNS AFTER THE STREAM HAS FINISHED.
 * Fitting W (the PCA of Section 3.3, an eigen-decomposition) is not part of this library.
 */
dresd_status dresd_fit_zscore(const void *sample, int64_t N, int d_in, dresd_dtype dtype, float *out_mean,
                              float *out_var, void *stream);

/*
 * Quantised candidate search.  The paper searches its datastore with an approximate
 * nearest-neighbour library (Section 3.5); the counterpart here scores an 8-bit copy of
 * the keys -- half the bytes of a 16-bit store, so about twice the queries per second of
 * the memory-bound exact scan -- and re-ranks the best candidates exactly.  Every step is
 * defined exactly (E4M3: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, largest
 * finite value 448; conversions round to nearest even and saturate):
 *
 *     k8[i][j] = e4m3(256 k[i][j])
 *     h1[j] = e4m3(256 q[j]),   h2[j] = e4m3(16 (256 q[j] - h1[j]))      q = unit query
 *     a[i]  = sum_j (h1[j] + h2[j] / 16) k8[i][j] / 65536                 approximate score
 *
 * The `candidates` rows with the largest a[i] (ties to the lower row) are scored exactly
 * against the 16-bit keys (fp32) and the top_n best of them returned like dresd_retrieve().
 * The result is NOT always the exact top_n: a true neighbour whose approximate score falls
 * below the candidate cut is missed; how often depends on `candidates` and on how close the
 * neighbours' scores lie (recall = the share of dresd_retrieve()'s rows that come back).
 *
 * dresd_quantise_keys       keys: device [N][d] fp16/bf16, d a multiple of 16; out_q8: device
 *                           [N][d] bytes; both 16-byte aligned.  Asynchronous on `stream`.
 * dresd_store_attach_quantised   the 8-bit copy of the store's keys (borrowed until destroy);
 *                           a set-up call, may allocate.  16-bit stores with d <= 2048.
 * dresd_retrieve_quantised  as dresd_retrieve_filtered() plus `candidates` in top_n .. DRESD_MAX_TOP_N:
 *                           first_tokens NULL (or -1 per query) = no first-token filter; with it only
 *                           keys whose first stored token matches are candidates (Section 3.5), and
 *                           missing neighbours are id -1, score -inf, tokens -1.
 *                           Asynchronous on `stream`; no allocation.
 */
dresd_status dresd_quantise_keys(const void *keys, int64_t N, int d, dresd_dtype dtype, void *out_q8, void *stream);
dresd_status dresd_store_attach_quantised(dresd_store *store, const void *keys_q8);
dresd_status dresd_retrieve_quantised(dresd_store *store, const void *queries, const int32_t *first_tokens, int B,
                                      int top_n, int draft_len, int candidates, int32_t *out_ids, float *out_scores,
                                      int32_t *out_tokens, void *stream);

/*
 * Process-wide switches (not part of the paper; for measurement and tests).
 *   "build_keys_pairs"  1 (default): dresd_build_keys runs on CTA pairs -- clusters of two
 *                       CTAs, one tensor-core instruction spanning both SMs, each CTA staging
 *                       half of the weight slab; 0: one CTA per tile.  Results are identical.
 *   "build_keys_wait_ms"  bound of the device-side waits of dresd_build_keys in milliseconds
 *                       (0 = default, about 2 s).
 *   "build_keys_debug_lose_stage"  test hook: in the next dresd_build_keys calls the first CTA (the
 *                       leader of the first pair) never receives the copies of pipeline stage
 *                       (value-1), so its waits run out: the kernel returns in an orderly way and
 *                       the call returns DRESD_ERR_TIMEOUT.  0 = off.
 * Unknown names and values outside the stated set return DRESD_ERR_INVALID.
 */
dresd_status dresd_set_global_option(const char *name, int value);

/*
 * Exchange step of a datastore whose rows are sharded over P GPUs.  Eq. 3 is an arg
 * max over the whole datastore; with the rows split into disjoint shards, the top_n
 * of the whole is the top_n of the union of the shards' top_n.  Each shard runs
 * dresd_retrieve() on its own rows; the P results (B * top_n * (8 + 4 draft_len) bytes
 * per shard) are gathered on one device -- NCCL all-gather, or peer copies -- and
 * this call merges them.
 *
 *   ids, scores, tokens  device, [P][B][top_n] / [P][B][top_n] / [P][B][top_n][draft_len]:
 *                        the shards' outputs, ids LOCAL to each shard (-1 = missing)
 *   row_offsets          device, int64 [P]: global row index of each shard's row 0,
 *                        ascending.  Output ids are int32: the shards may hold at most
 *                        2^31 - 1 rows in all (offset + rows of every shard <= 2^31 - 1);
 *                        the call cannot see the shards' sizes, so the caller checks this
 *                        where the offsets are made
 *   out_*                as for dresd_retrieve(), ids global.
 */
dresd_status dresd_merge_shards(const int32_t *ids, const float *scores, const int32_t *tokens,
                                const int64_t *row_offsets, int P, int B, int top_n, int draft_len,
                                int32_t *out_ids, float *out_scores, int32_t *out_tokens, void *stream);

/*
 * The same merge for results that were exchanged in ONE all-gather (the message is
 * latency-bound: 480 bytes per shard at B = 1, n = 10, L = 10): shard p's block
 * of B * top_n * (2 + draft_len) 32-bit words is
 *     ids [B][top_n] int32 | scores [B][top_n] fp32 | tokens [B][top_n][draft_len] int32
 * and `packed` (device) holds the P blocks back to back, as an all-gather of the
 * blocks leaves them.  Everything else as for dresd_merge_shards().
 */
dresd_status dresd_merge_shards_packed(const int32_t *packed, const int64_t *row_offsets, int P, int B,
                                       int top_n, int draft_len, int32_t *out_ids, float *out_scores,
                                       int32_t *out_tokens, void *stream);

/*
 * The same call for callers whose queries and results live in HOST memory, and
 * waits for `stream`.  When all four buffers are page-locked and mapped (e.g.
 * cudaHostAlloc, cudaHostRegister, a pinned framework tensor), the kernels read the
 * queries and write the results across the bus themselves (B * d_in elements in,
 * B * top_n * (8 + 4 draft_len) bytes out) and no copy is enqueued; otherwise the
 * queries are copied to a staging buffer and the three results copied back.  The
 * datastore itself stays on the device.  Returns the device status word as well.
 */
dresd_status dresd_retrieve_host(dresd_store *store, const void *queries_host, int B, int top_n,
                                 int draft_len, int32_t *out_ids_host, float *out_scores_host,
                                 int32_t *out_tokens_host, void *stream);

/*
 * Eq. 1 -> Section 3.3 -> Eq. 2 alone: writes the unit-length queries,
 * fp32 [B][d] (device), exactly as the scoring kernels consume them.
 */
dresd_status dresd_preprocess(dresd_store *store, const void *queries, int B, float *out_qhat,
                              void *stream);

/*
 * Device-side health: every wait inside the kernels is bounded; a wait that
 * expires records DRESD_ERR_TIMEOUT in a device word and the kernel returns.
 * This call synchronises the store's last stream and reports (then clears)
 * that word: DRESD_OK or DRESD_ERR_TIMEOUT.
 */
dresd_status dresd_store_status(dresd_store *store);

/*
 * Bounds-checked debug build.  The library is also built as libdresd_debug.so with
 * -DDRESD_DEBUG_BOUNDS (the Python binding loads it when the environment variable
 * DRESD_DEBUG is 1): every global index and pipeline-ring slot that the kernels form -- stage
 * slots and tile coordinates of the loaders, rows of the first-token column, entries of the
 * window table, positions in the candidate array, the row ids of candidates and winners -- is
 * checked where it is formed; a violation skips the access and records its site in the status
 * word, and dresd_store_status() then returns DRESD_ERR_INTERNAL with the site number in the
 * message.  It stands in for a memory checker on systems where none can be run; it is a few per
 * cent slower and otherwise computes the same results.
 *   dresd_debug_build()            1 in the debug build, 0 in the release build.
 *   dresd_store_debug_selftest()   debug build: one thread fails check 7 on purpose (no access is
 *                                  attempted), so that the reporting path can be seen to work;
 *                                  release build: DRESD_ERR_UNSUPPORTED.
 */
int dresd_debug_build(void);
dresd_status dresd_store_debug_selftest(dresd_store *store, void *stream);

/*
 * Kernel-selection knobs for tests and measurements (set between calls).
 *   "scan_path"  0 = automatic, 1 = CUDA-core/mma.sync streaming kernel,
 *                2 = tcgen05 tensor-core kernel (16-bit keys only).
 *   "grid"       CTAs of the scoring kernel, 0 = one per SM.
 *   "probe"      large batches on large stores first run a probe pass over every
 *                value-th key tile to seed the selection filter; 0 = never,
 *                1 (default) = a stride that follows the call: 64 (64 queries x top-32) to 256
 *                (few results), less on a small store (at least one probe tile per CTA, no probe
 *                pass below eight tiles per CTA).
 *   "pack2"      1 (default): 64-byte keys are scanned as rows of two keys (one 128-byte line) --
 *                the 8-bit copy of a store with d = 64 in the quantised search (up to 32 queries
 *                per call), and a 16-bit store with d = 32 and an even number of rows in the exact
 *                search (up to 16 queries per call); 0 = one key per row.  Results do not change.
 *   "keys_as_m"  0 (default): batches of 17-64 queries on rows of 129-256 elements run the
 *                tcgen05 kernel with the queries as the M = 128 and the keys as the
 *                N = 256 operand of the instruction; 1 = keys as the M operand at every
 *                batch size (the form all other shapes use).  Results do not change.
 *   "merged_columns"  0 (default): batches of 33-64 queries on rows of at most 64 elements run the
 *                tcgen05 kernel with ONE accumulator column per query (both 16-bit terms of the query
 *                are accumulated into the same column, scaled by a power of two; half the columns to
 *                compare per key, twice the instructions); 1 = that form for every batch of more
 *                than 16 queries that the keys-as-N form does not take, 2 = never.  Scores agree with
 *                the two-column form to fp32 accumulation order (last bits), within the tolerances.
 *   "merge_level"  0 (default, = 24): the tcgen05 kernels fold a query's queue of 32 candidates into its
 *                sorted list once it holds this many (1..32).  Results do not change.
 *   "epi_warps"  0 (default): the forms for 33-64 queries with several sub-tiles per tile (one column
 *                per query on one-slab rows; two columns per query on rows of two slabs and on rows
 *                wider than 256) run sixteen selection warps; 8 = eight, as every other form.
 *                Results do not change.
 *   "round_per_tile"  0 (default): the selection warps of the tcgen05 kernel with the keys as M fold
 *                their candidate queues in rounds held on demand; 1 = a round after every tile (the
 *                earlier form; token windows and the probe pass always use it).  Results do not change.
 *   "fast_reject"  1 (default): the kernel with the keys as N tests a unit of 16 scores with packed
 *                sign-bit arithmetic before the exact compare; 0 = exact compare only.  Results do not change.
 *   "first_token_windows"  1 (default): on a store indexed by dresd_store_index_first_tokens()
 *                filtered calls scan only the rows of their queries' tokens; 0 = scan every row.
 *                Results do not change.
 *   "wait_ms"    bound of the device-side waits of the scoring kernels in
 *                milliseconds (0 = default, about 2 s).
 *   "debug_lose_stage"  test hook: in the next calls the first CTA of the scoring kernel
 *                (whichever kernel the call selects) never receives the copies of pipeline
 *                stage (value-1), so its waits run out: the kernel returns in an orderly way,
 *                frees its tensor memory, and dresd_store_status() reports
 *                DRESD_ERR_TIMEOUT; the results of such a call are incomplete.  0 = off.
 *   "debug_no_select"  measurement hook: the tcgen05 scoring kernel streams and scores
 *                every key but lets nothing pass its filter (results are empty); the
 *                time of such a call is the floor against which the cost of
 *                selection, merge and gather is measured.  0 = off.
 *   "profile"    > 0: record a CUDA-event pair around the scoring kernel(s) of
 *                each of the next `value` dresd_retrieve() calls (see
 *                dresd_store_profile_read); 0 = off (default).
 *   "profile_stride"  k >= 1 (default 1): while "profile" is armed, only every k-th call is
 *                timed.  The events sit between the kernels of a call and hold up the overlap
 *                of one kernel's set-up with its predecessor's tail, so a sparse sample
 *                disturbs a throughput measurement less.
 * Unknown names return DRESD_ERR_INVALID.
 */
dresd_status dresd_store_set_option(dresd_store *store, const char *name, int value);

/*
 * Waits for the store's last stream, then returns the summed device time (ms)
 * of the scoring kernel (Eq. 3 over every key, with the fused selection) over
 * the profiled calls since the last read, and how many calls that covers.
 * Resets the counter so that profiling continues with fresh slots.
 */
dresd_status dresd_store_profile_read(dresd_store *store, double *scan_ms_total, int *calls);

/* Number of kernels dresd_retrieve() enqueued in the store's last call. */
int dresd_store_last_launches(const dresd_store *store);

/* Passes over the key matrix made by the store's last dresd_retrieve(): 1 per scoring
 * launch over all keys, plus 1/stride when the probe pass ran. */
double dresd_store_last_key_passes(const dresd_store *store);

/* Message of the calling thread's last failing call ("" if none). */
const char *dresd_last_error(void);

/*
 * (No counterpart in the paper: a deployment variant of dresd_retrieve().)
 *
 * Retrieval for callers that cannot allocate device memory when they need a
 * draft -- a serving runtime that gave all device memory to its own pool and
 * forbids cudaMalloc afterwards, a plug-in living inside another program's
 * memory budget, a latency-critical path that cannot afford the device-wide
 * synchronisation an allocation implies.  dresd_store_create() needs cudaMalloc
 * for its workspace; this call needs no store: its workspace (unit queries,
 * their 16-bit split, per-CTA candidate lists, status word) is a fixed
 * ~576 KB array inside the library image, held by every GPU that loads the
 * library until the process exits.  It calls no cudaMalloc/cudaFree and no
 * allocating library routine; it computes what dresd_retrieve() computes
 * on a store without z-scoring or projection (Eq. 2, Eq. 3, Section 3.5).
 * fp32 stores run the kernel dresd_retrieve() runs.  16-bit stores run the
 * STREAMING scoring kernel (the one store option "scan_path" 1 selects), not the
 * tcgen05 kernel that dresd_retrieve() uses by default: its workspace is smaller
 * and it needs no query-operand descriptor.  Both accumulate in fp32 and meet the
 * same tolerances, but in a different order, so against the default store path
 * scores can differ in the last bits and rows that tie within that rounding can
 * swap; against a store with "scan_path" 1 results are identical.
 *
 *   keys, next_tokens, N, d, dtype, stored_len   as for dresd_store_create();
 *   queries [B][d], B, top_n, draft_len, out_*   as for dresd_retrieve()
 *   (all device pointers; the caller owns inputs and outputs).
 *
 * Limits: B <= DRESD_NOALLOC_MAX_BATCH (8); larger B returns
 * DRESD_ERR_UNSUPPORTED with a message, as do top_n > DRESD_MAX_TOP_N and
 * d > DRESD_MAX_DIM.  Pointers are checked for NULL and alignment only.
 *
 * The first call on each device resolves the workspace's device address
 * (with that device current); make that first call outside any stream
 * capture.  The workspace is ONE per device and keeps the previous call's
 * contents (the call clears the one word that must start at zero): two calls
 * whose kernels overlap on the GPU -- different streams, or threads -- race
 * on it and return garbage.  Serialise them on one stream.  Asynchronous on
 * `stream` like dresd_retrieve().
 *
 * dresd_noalloc_status() is dresd_store_status() for this call: it waits for
 * `stream`, reads the workspace's status word with a 4-byte copy (no allocation
 * either) and returns DRESD_OK, or DRESD_ERR_TIMEOUT when a bounded device-side
 * wait of the last call expired (the word is then cleared).  Call it after a
 * dresd_retrieve_noalloc() and before the next one, which resets the word.
 */
enum { DRESD_NOALLOC_MAX_BATCH = 8 };
dresd_status dresd_retrieve_noalloc(const void *keys, const int32_t *next_tokens, int64_t N, int d,
                                    dresd_dtype dtype, int stored_len, const void *queries, int B,
                                    int top_n, int draft_len, int32_t *out_ids, float *out_scores,
                                    int32_t *out_tokens, void *stream);
dresd_status dresd_noalloc_status(void *stream);

/* Frees the workspace only, never caller memory.  NULL is allowed. */
void dresd_store_destroy(dresd_store *store);

#ifdef __cplusplus
}
#endif
#endif /* DRESD_H */

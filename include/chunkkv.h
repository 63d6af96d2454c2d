/*
 * chunkkv.h - C ABI of the ChunkKV prefill-time KV-cache compression library (CUDA, sm_100a).
 *
 * The operation (ChunkKV paper, Algorithm 3 "ChunkKV Implementation", with Algorithm 1 for the
 * notation and Algorithm 2 for layer-wise index reuse), for one layer and each KV head h:
 *
 *   P = L - w                      prefix length; the last w rows are the observation window
 *   R = w * (Hq / Hkv)             window queries of the Hq/Hkv query heads sharing KV head h
 *   p[i, j]                        softmax over the keys row i can see of q_i . k_j / sqrt(d);
 *                                  row (g, r) sits at position P + r and sees key j iff j <= P + r
 *   t[j]   = sum_i p[i, j]         token score, j in [0, P)
 *   C      = ceil(P / c)           chunks over the prefix (origin 0, stride c, last one clipped)
 *   s[ch]  = sum_{j in chunk} t[j] chunk score
 *   k      = min(floor((budget - w) / c), C)
 *   keep the k chunks with the largest s (ties: lower chunk id), whole chunks, plus the window
 *   idx    = kept token positions in ascending order (window last), padded with -1 to
 *            n_max = k * c + w
 *   out_K[n] = K[idx[n]], out_V[n] = V[idx[n]]  (bit copies; zero rows where idx is -1)
 *
 * Conventions shared by every entry point
 *   - All tensor pointers are DEVICE pointers (unless a name says host), 16-byte aligned,
 *     dense row-major, owned by the caller, and must stay valid until the work queued on
 *     `stream` has finished. bf16 tensors are passed as `const void*`.
 *       q_obs [Hq, w, d] bf16   queries of the last w positions (after positional encoding);
 *                               query head g belongs to KV head g / (Hq / Hkv)
 *       K, V  [Hkv, L, d] bf16  keys / values of the layer, window rows included
 *       token scores [Hkv, P] f32, chunk scores [Hkv, C] f32
 *       idx   [Hkv, n_max] int32, out_K / out_V [Hkv, n_max, d] bf16
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream). Calls only
 *     enqueue work; they never synchronise the device (except where stated).
 *   - Limits: d in {64, 128}; Hq a multiple of Hkv; R = w * Hq / Hkv <= 256; 1 <= w <= L;
 *     c >= 1; budget >= w; Hkv * L < 2^23 (8 M keys per layer).
 *   - Return value: CHUNKKV_OK (0) or a negative CHUNKKV_E* code. Arguments are checked on
 *     the host before anything is launched; nothing is thrown and nothing aborts.
 *   - Scratch memory: scoring needs device scratch of chunkkv_workspace_bytes(...) bytes. The
 *     library never allocates and never frees: the caller hands it a buffer once with
 *     chunkkv_set_workspace (a set-up call), and every entry point that scores returns
 *     CHUNKKV_ENOWORKSPACE while no buffer, or too small a buffer, is set. Calls that use the
 *     scratch of one device must be ordered on the GPU (same stream, or otherwise serialised):
 *     concurrent calls would share it. Lanes and pipes (below) take their scratch per object.
 */
#ifndef CHUNKKV_H_
#define CHUNKKV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define CHUNKKV_API __attribute__((visibility("default")))
#else
#define CHUNKKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define CHUNKKV_OK              0
#define CHUNKKV_EINVAL_NULL    -1  /* a required pointer is NULL */
#define CHUNKKV_EINVAL_SHAPE   -2  /* a size violates the limits above */
#define CHUNKKV_EINVAL_ALIGN   -3  /* a tensor pointer is not 16-byte aligned */
#define CHUNKKV_ENOWORKSPACE   -4  /* no workspace set (chunkkv_set_workspace), or too small for the shape */
#define CHUNKKV_ECUDA          -5  /* a CUDA runtime or driver call failed (see chunkkv_last_cuda_error) */
#define CHUNKKV_EDEVICE        -6  /* a kernel gave up on a bounded wait (see chunkkv_device_status) */
#define CHUNKKV_ETOOLARGE      -7  /* the problem needs more scratch than a fixed-size variant provides */

/* Human-readable name of a status code (static string, never NULL). */
CHUNKKV_API const char* chunkkv_strerror(int status);

/* The cudaError_t (as int) recorded by the most recent CHUNKKV_ECUDA on this thread. */
CHUNKKV_API int chunkkv_last_cuda_error(void);

/* C = ceil((L - w) / c); 0 when L == w. Negative status on invalid sizes. (Algorithm 3, chunk count.) */
CHUNKKV_API int chunkkv_num_chunks(int L, int w, int c);

/* k = min(floor((budget - w) / c), C). (Algorithm 3, "Limit k to available chunks".) */
CHUNKKV_API int chunkkv_num_kept_chunks(int L, int w, int c, int budget);

/* n_max = k * c + w: row count of idx / out_K / out_V per head. */
CHUNKKV_API int chunkkv_out_len(int L, int w, int c, int budget);

/* Bytes of device scratch that scoring a layer of this shape needs (0 on invalid sizes). */
CHUNKKV_API size_t chunkkv_workspace_bytes(int L, int Hq, int Hkv, int d, int w, int c);

/*
 * Set-up: use caller-owned device memory (256-byte aligned, on the current device) as scratch for
 * all later calls on this device. Its first 256 bytes hold the library's device status word and
 * hand-over counters and are cleared by this call. This is the one call that synchronises the
 * device (work queued earlier may still be using the previous buffer). Passing (NULL, 0) detaches
 * the buffer. The caller keeps ownership and must keep the buffer alive while calls may use it.
 */
CHUNKKV_API int chunkkv_set_workspace(void* dev_ptr, size_t bytes);

/*
 * Synchronise `stream`, then report whether any kernel of this library on the current device
 * abandoned a bounded wait since the last call (CHUNKKV_EDEVICE) - a defect report, not an
 * expected outcome. Clears the status word.
 */
CHUNKKV_API int chunkkv_device_status(void* stream);

/*
 * Steps "observe-window attention scores" and "chunk score calculation" (Algorithm 3; Algorithm 1
 * "Observe Window Calculation" / "Chunk Attention Score Calculation").
 *   out_chunk_scores [Hkv, C] f32   required
 *   out_token_scores [Hkv, P] f32   optional (NULL to skip); computed by a second pass of the
 *                                   same kernels with chunk size 1, so it costs scratch for
 *                                   chunk size 1 as well
 * With P == 0 nothing is written.
 */
CHUNKKV_API int chunkkv_score(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d, int w, int c,
                  float* out_token_scores, float* out_chunk_scores, void* stream);

/*
 * chunkkv_score for callers that must not allocate. (No counterpart in the paper: this is a
 * deployment convenience, not a step of the method.)
 *
 * Who needs it: serving processes that hand every free byte of HBM to their own cache pool at
 * start-up and therefore have no buffer left to pass to chunkkv_set_workspace later, and callers
 * that cannot reach an allocator at all (a plug-in that only sees raw pointers). This entry point
 * calls no cudaMalloc, cudaFree or any other allocating routine, and ignores
 * chunkkv_set_workspace: its scratch is a fixed 8 MiB array that lives in the library's device
 * image (every GPU on which this entry point has been called holds those 8 MiB until the process
 * exits).
 *
 * Same arguments, layouts and result as chunkkv_score without the token-score output:
 * out_chunk_scores [Hkv, C] f32. Shapes whose chunkkv_workspace_bytes(L, Hq, Hkv, d, w, c)
 * exceeds 8 MiB are rejected with CHUNKKV_ETOOLARGE, shapes outside the library's limits with
 * CHUNKKV_EINVAL_SHAPE, and nothing is launched.
 *
 * The first call on each device looks up the device address of the array (with that device
 * current). The CUDA runtime loads device code lazily, so that first call is also the moment the
 * array takes its 8 MiB: make one warm-up call per device at start-up, before the process gives
 * its free memory away and outside any stream capture. Later calls leave the amount of free
 * device memory unchanged. All calls on a device share the one array, which keeps whatever the
 * previous call left in it; nothing in it needs clearing between calls, and calls that overlap on
 * the GPU (different streams, no ordering) race on it - order them.
 *
 * chunkkv_score_noalloc_status synchronises `stream`, then reports whether a kernel launched by
 * chunkkv_score_noalloc on the current device abandoned a bounded wait since the last status call
 * (CHUNKKV_EDEVICE; out_chunk_scores of that call are then incomplete) and clears the mark.
 * chunkkv_device_status does not cover this entry point.
 */
CHUNKKV_API int chunkkv_score_noalloc(const void* q_obs, const void* K, int L, int Hq, int Hkv, int d,
                                      int w, int c, float* out_chunk_scores, void* stream);
CHUNKKV_API int chunkkv_score_noalloc_status(void* stream);

/*
 * Step "top-k chunk selection" and the kept-index list (Algorithm 3: Top-K, selection mask,
 * window forced on, nonzero). chunk_scores [Hkv, C] f32 -> out_idx [Hkv, n_max] int32:
 * ascending token positions of the k best chunks (ties to the lower chunk id), then P..L-1,
 * then -1 padding (only when the clipped last chunk is among the kept ones).
 */
CHUNKKV_API int chunkkv_select(const float* chunk_scores, int L, int Hkv, int w, int c, int budget,
                   int32_t* out_idx, void* stream);

/*
 * Step "compression" (Algorithm 3 / Algorithm 2: index_select on K and on V).
 * idx [Hkv, n_max] int32 -> out_K, out_V [Hkv, n_max, d]; entries outside [0, L) give zero rows.
 * out_K/out_V must not overlap K/V.
 */
CHUNKKV_API int chunkkv_gather(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d,
                   int n_max, void* out_K, void* out_V, void* stream);

/*
 * The whole layer (Algorithm 3), or - with reuse_idx non-NULL - a layer that reuses another
 * layer's indices (Algorithm 2, else-branch): scoring and selection are skipped, reuse_idx
 * [Hkv, n_max] is copied to out_idx (they may be the same buffer) and only the gather runs.
 */
CHUNKKV_API int chunkkv_compress_layer(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                           int d, int w, int c, int budget, const int32_t* reuse_idx_or_null,
                           void* out_K, void* out_V, int32_t* out_idx, void* stream);

/*
 * Adapters to the steps either side of the path (the paper runs the compression at the end of
 * prefill - "q_observe <- Q[T_q - w : T_q]" in Algorithm 3 takes the last w queries of the layer -
 * and hands the compacted cache to decoding).
 *
 * chunkkv_window_queries: q_obs [Hq, w, d] bf16 out of the layer's fused QKV projection output
 *   qkv [T, row_elems] bf16 (token-major; the Hq query heads first in a row, then keys and values;
 *   row_elems >= (Hq + 2 Hkv) d, a multiple of 8; values before the rotary position embedding).
 *   The window is the last w rows. cos_rows / sin_rows [w, d / 2] f32 are the embedding-table rows
 *   of the window's positions; element i is paired with element i + d / 2 (rotate-half):
 *   out[i] = x[i] cos[i] - x[i + d/2] sin[i], out[i + d/2] = x[i + d/2] cos[i] + x[i] sin[i],
 *   computed in fp64 and rounded once (through fp32) to bf16. All pointers are device memory.
 *
 * chunkkv_gather_paged: chunkkv_gather with a paged destination. cache_K / cache_V
 *   [num_pages, page_size, Hkv, d] bf16; compacted position n of every head goes to page
 *   block_table[n / page_size] (device int32, ceil(n_max / page_size) entries), slot n % page_size;
 *   zero rows where idx is outside [0, L). Entries of the block table outside [0, num_pages) are
 *   skipped. Pages not named and slots past n_max stay as they are.
 *
 * chunkkv_compress_layer_paged: chunkkv_compress_layer (or, with reuse_idx, a layer that reuses
 *   indices) writing the kept rows to a paged cache instead of dense out_K / out_V; out_idx
 *   [Hkv, n_max] is still written. The one-launch layer kernel places the rows through the block table
 *   where the shape fits it; otherwise separate score / select / gather launches.
 *
 * chunkkv_compress_layer_strided: chunkkv_compress_layer (or, with reuse_idx, a layer that reuses
 *   indices) on keys and values that are not packed [Hkv, L, d]: row l of head h of K starts at
 *   element l * k_token_stride + h * k_head_stride of K (likewise V); a token-major prefill cache
 *   [L, Hkv, d] has token stride Hkv * d and head stride d. Strides are in bf16 elements, multiples
 *   of 8 and at least d; K and V 16-byte aligned. The outputs are packed as usual. With the packed
 *   strides (d and L * d) this is chunkkv_compress_layer itself; otherwise the one-launch layer kernel
 *   where the shape fits it (chunk sizes 10 and 20, up to 128 score rows per scoring head), else separate
 *   score / select / gather launches. Returns CHUNKKV_EINVAL_SHAPE for other strides.
 */
CHUNKKV_API int chunkkv_window_queries(const void* qkv, long long row_elems, int T, int Hq, int Hkv, int d, int w,
                                       const float* cos_rows, const float* sin_rows, void* out_q_obs, void* stream);
CHUNKKV_API int chunkkv_gather_paged(const void* K, const void* V, const int32_t* idx, int L, int Hkv, int d, int n_max,
                                     const int32_t* block_table, int page_size, int num_pages, void* cache_K,
                                     void* cache_V, void* stream);
CHUNKKV_API int chunkkv_compress_layer_paged(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                                             int d, int w, int c, int budget, const int32_t* reuse_idx_or_null,
                                             const int32_t* block_table, int page_size, int num_pages, void* cache_K,
                                             void* cache_V, int32_t* out_idx, void* stream);
CHUNKKV_API int chunkkv_compress_layer_strided(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                                               int d, int w, int c, int budget, long long k_token_stride,
                                               long long k_head_stride, long long v_token_stride,
                                               long long v_head_stride, const int32_t* reuse_idx_or_null,
                                               void* out_K, void* out_V, int32_t* out_idx, void* stream);

/*
 * A whole model with layer-wise index reuse (Algorithm 2): layer l computes its indices iff
 * l mod reuse_depth == 0 (Algorithm 3 on q_obs[l], K[l], V[l]); every other layer gathers with the
 * indices of layer floor(l / reuse_depth) * reuse_depth, which are also copied to its out_idx.
 * All layers share L, Hq, Hkv, d, w, c and budget.
 *   q_obs, K, V, out_K, out_V, out_idx   HOST arrays of n_layers DEVICE pointers (layouts as in
 *                                        chunkkv_compress_layer); q_obs[l] may be NULL for layers
 *                                        that reuse indices. The arrays are read during the call
 *                                        only. Output buffers of different layers must not overlap.
 * Same results as the corresponding sequence of chunkkv_compress_layer calls. Where the shape
 * allows (chunk size 10 or 20, at most 128 query rows per KV head or an even number of grouped query
 * heads, key range per SM within tensor memory) the layers run through one persistent kernel per
 * group of up to 32 layers in which scoring layer l + 1 overlaps selecting and gathering layer l;
 * otherwise they run layer by layer. Needs a workspace of chunkkv_model_workspace_bytes(...) bytes
 * (chunkkv_set_workspace); returns CHUNKKV_ENOWORKSPACE otherwise. Queued on `stream`; the calls of
 * one device that use the workspace must be ordered.
 */
CHUNKKV_API size_t chunkkv_model_workspace_bytes(int n_layers, int L, int Hq, int Hkv, int d, int w, int c,
                                                 int budget, int reuse_depth);
CHUNKKV_API int chunkkv_compress_model(int n_layers, const void* const* q_obs, const void* const* K,
                                       const void* const* V, int L, int Hq, int Hkv, int d, int w, int c,
                                       int budget, int reuse_depth, void* const* out_K, void* const* out_V,
                                       int32_t* const* out_idx, void* stream);

/*
 * chunkkv_compress_model on keys and values that are not packed [Hkv, L, d] (the same strides, in bf16
 * elements, for every layer: see chunkkv_compress_layer_strided; a token-major cache [L, Hkv, d] has
 * token stride Hkv * d and head stride d). Outputs are packed. The persistent kernel scores through
 * tensor maps with those strides and copies the kept rows one row at a time; shapes it does not take
 * run layer by layer. No counterpart in the paper: it is Algorithm 2 on another memory layout.
 */
CHUNKKV_API int chunkkv_compress_model_strided(int n_layers, const void* const* q_obs, const void* const* K,
                                               const void* const* V, int L, int Hq, int Hkv, int d, int w, int c,
                                               int budget, int reuse_depth, long long k_token_stride,
                                               long long k_head_stride, long long v_token_stride,
                                               long long v_head_stride, void* const* out_K, void* const* out_V,
                                               int32_t* const* out_idx, void* stream);

/*
 * chunkkv_compress_model writing every layer's kept rows into that layer's paged decode cache
 * (cache_K[l] / cache_V[l] [num_pages, page_size, Hkv, d] through block_tables[l], as in
 * chunkkv_gather_paged; one page_size and num_pages for all layers); out_idx[l] [Hkv, n_max] is still
 * written. Runs layer by layer through chunkkv_compress_layer_paged (the one-launch layer kernel places
 * the rows through the block table with all its threads), in Algorithm 2's order.
 */
CHUNKKV_API int chunkkv_compress_model_paged(int n_layers, const void* const* q_obs, const void* const* K,
                                             const void* const* V, int L, int Hq, int Hkv, int d, int w, int c,
                                             int budget, int reuse_depth, const int32_t* const* block_tables,
                                             int page_size, int num_pages, void* const* cache_K, void* const* cache_V,
                                             int32_t* const* out_idx, void* stream);

/*
 * Algorithm 1's budget rule, as an alternative to Algorithm 3's (which the calls above follow):
 * k = floor(L_max / c) chunks are selected (at most the C that exist), their tokens are taken in
 * ascending order and cut to the first L_max - w ("K'[0 : L_max - w]"), and the observe window
 * takes the last w places. `budget` is L_max. chunkkv_budget_from_ratio gives L_max for the
 * compression ratios of the paper's experiments: floor(ratio * L), ratio in [0, 1].
 * chunkkv_out_len_alg1 = min(k * c, L_max - w) + w is the row count n_max of out_idx / out_K /
 * out_V for these two calls; a kept clipped last chunk leaves -1 / zero-row padding at the end.
 * Chunk grid, tie-break, layouts, ownership and error codes are those of chunkkv_select and
 * chunkkv_compress_layer (no index reuse argument: reuse layers call chunkkv_compress_layer or
 * chunkkv_gather with these indices). Scoring, selection and gathering run as three launches.
 */
CHUNKKV_API int chunkkv_budget_from_ratio(int L, double ratio);
CHUNKKV_API int chunkkv_num_kept_chunks_alg1(int L, int w, int c, int budget);
CHUNKKV_API int chunkkv_out_len_alg1(int L, int w, int c, int budget);
CHUNKKV_API int chunkkv_select_alg1(const float* chunk_scores, int L, int Hkv, int w, int c, int budget,
                        int32_t* out_idx, void* stream);
CHUNKKV_API int chunkkv_compress_layer_alg1(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                                int d, int w, int c, int budget, void* out_K, void* out_V, int32_t* out_idx,
                                void* stream);

/*
 * Index similarity between two layers (the paper's section on layer-wise index reuse reports the
 * Jaccard similarity of the preserved indices of adjacent layers; Algorithm 2 shares indices
 * because it is high). Per KV head h: out_ratio[h] = |A n B| / |A u B| (1 when both are empty),
 * A and B the valid (non-negative) entries of row h of idx_a [Hkv, n_a] and idx_b [Hkv, n_b].
 * Rows must be as chunkkv_select / chunkkv_compress_layer write them: ascending, no repeats,
 * -1 padding last. out_counts [Hkv, 3] int32 (optional, may be NULL) receives |A n B|, |A|, |B|.
 * All pointers are device memory; the call is queued on `stream`.
 */
CHUNKKV_API int chunkkv_jaccard(const int32_t* idx_a, const int32_t* idx_b, int Hkv, int n_a, int n_b,
                                float* out_ratio, int32_t* out_counts, void* stream);

/*
 * Lanes: several layers in flight at once (Algorithm 2 visits the layers one after another, and
 * they are independent). A lane is caller-owned scratch plus a CTA budget. Layers submitted to
 * different lanes on different streams run concurrently, each on its share of the SMs, so the
 * latency-bound steps of one layer (top-k selection, grid-wide hand-overs) overlap the
 * bandwidth-bound scoring and gathering of the others.
 *
 *   chunkkv_lane_bytes          scratch a lane needs for a shape with a CTA budget (0 = all SMs)
 *   chunkkv_lane_init           clears the lane's 256-byte header (queued on `stream`); call once
 *                               before first use, and again before using the lane with a different
 *                               CTA budget
 *   chunkkv_compress_layer_lane chunkkv_compress_layer with the lane's scratch and at most
 *                               max_ctas CTAs (0 = all SMs). Calls on one lane must be ordered
 *                               (same stream). The budgets of all lanes that may run at the same
 *                               time must add up to no more than the number of SMs: the layer
 *                               kernel synchronises its CTAs grid-wide, which needs all of them
 *                               resident. With a budget of at most half the SMs the rows are
 *                               gathered by a second launch on the same stream whose small CTAs
 *                               run on every SM beside the other lanes' resident CTAs.
 *   chunkkv_lane_status         synchronises `stream`, then CHUNKKV_OK or CHUNKKV_EDEVICE for the
 *                               lane (and clears its header)
 * lane must be 256-byte aligned device memory.
 */
CHUNKKV_API size_t chunkkv_lane_bytes(int L, int Hq, int Hkv, int d, int w, int c, int max_ctas);
CHUNKKV_API int chunkkv_lane_init(void* lane, size_t bytes, void* stream);
CHUNKKV_API int chunkkv_lane_status(void* lane, void* stream);
CHUNKKV_API int chunkkv_compress_layer_lane(const void* q_obs, const void* K, const void* V, int L, int Hq, int Hkv,
                                            int d, int w, int c, int budget, const int32_t* reuse_idx_or_null,
                                            void* out_K, void* out_V, int32_t* out_idx,
                                            void* lane, size_t lane_bytes, int max_ctas, void* stream);

/*
 * Pipes: a lane whose row gathers overlap the next layer. Scoring and selecting a layer
 * (Algorithm 3 up to the indices) is bound by arithmetic on the lane's SMs; gathering its rows
 * is bound by memory traffic and needs none of the lane's scratch. A pipe therefore runs the
 * lane's layer kernels of successive layers back to back on the caller's stream, with at most
 * max_ctas CTAs, and each layer's row gather on a stream of its own, in small CTAs that share SMs
 * with resident layer-kernel CTAs of this and other pipes.
 *
 *   chunkkv_pipe_bytes   device scratch a pipe needs for a shape and CTA budget (0 = all SMs);
 *                        the same as chunkkv_lane_bytes
 *   chunkkv_pipe_open    makes the host object (a side stream and two events) over caller-owned
 *                        scratch (256-byte aligned device memory, header cleared here); synchronous.
 *   chunkkv_pipe_layer   chunkkv_compress_layer (compute path, q_obs required) through the pipe:
 *                        the layer kernel is queued on `stream`, the gather on the pipe's stream.
 *                        Calls on one pipe must come from one thread and use one stream. The
 *                        outputs of a layer are complete only for work queued after
 *                        chunkkv_pipe_join; layers queued before the join must not share output
 *                        buffers with each other. The CTA budgets of pipes (and lanes) that may
 *                        run at the same time must add up to no more than the number of SMs.
 *   chunkkv_pipe_join    makes `stream` wait for everything the pipe has queued (device-side
 *                        wait, no host synchronisation). Required before the outputs are used
 *                        and before a stream capture that contains pipe calls ends.
 *   chunkkv_pipe_status  join + synchronise `stream`; CHUNKKV_OK or CHUNKKV_EDEVICE (an abandoned
 *                        wait in a layer kernel; the status word is cleared)
 *   chunkkv_pipe_close   waits for the pipe's stream and frees the host object (not the scratch)
 * Errors: CHUNKKV_ENOWORKSPACE when the scratch is too small for the shape; otherwise as
 * chunkkv_compress_layer. The paper runs its layers one after another (Algorithm 2); overlapping
 * them changes no result.
 */
CHUNKKV_API size_t chunkkv_pipe_bytes(int L, int Hq, int Hkv, int d, int w, int c, int max_ctas);
CHUNKKV_API int chunkkv_pipe_open(void* scratch, size_t bytes, int max_ctas, void** pipe_out);
CHUNKKV_API int chunkkv_pipe_layer(void* pipe, const void* q_obs, const void* K, const void* V, int L, int Hq,
                                   int Hkv, int d, int w, int c, int budget, void* out_K, void* out_V,
                                   int32_t* out_idx, void* stream);
CHUNKKV_API int chunkkv_pipe_join(void* pipe, void* stream);
CHUNKKV_API int chunkkv_pipe_status(void* pipe, void* stream);
CHUNKKV_API int chunkkv_pipe_close(void* pipe);

/*
 * End-to-end convenience for callers whose tensors live in (ideally pinned) HOST memory:
 * copies q_obs, K, V to the given device staging buffers, runs chunkkv_compress_layer and
 * copies out_K, out_V, out_idx back to the host buffers, all queued on `stream`.
 * host_* are host pointers; dev_* are device buffers of the same sizes.
 */
CHUNKKV_API int chunkkv_compress_layer_host(const void* host_q_obs, const void* host_K, const void* host_V,
                                int L, int Hq, int Hkv, int d, int w, int c, int budget,
                                void* dev_q_obs, void* dev_K, void* dev_V,
                                void* dev_out_K, void* dev_out_V, int32_t* dev_out_idx,
                                void* host_out_K, void* host_out_V, int32_t* host_out_idx,
                                void* stream);

/*
 * Optional per-kernel timing for benchmarks. While enabled, the entry points bracket each
 * kernel with CUDA events on the launching stream. chunkkv_profile_read synchronises the
 * device and returns, per kernel slot, accumulated milliseconds and launch counts since the
 * last read (arrays of CHUNKKV_PROFILE_SLOTS entries), then resets them.
 * Slots: 0 score (or the fused whole-layer kernel of chunkkv_compress_layer), 1 chunk-score
 * finalisation, 2 select, 3 gather.
 */
#define CHUNKKV_PROFILE_SLOTS 4
CHUNKKV_API int chunkkv_profile_enable(int on);
CHUNKKV_API int chunkkv_profile_read(float* ms_per_slot, int* launches_per_slot);

#ifdef __cplusplus
}
#endif
#endif /* CHUNKKV_H_ */

/*
 * libfocus -- the per-denoising-step sparse-attention path of Focus-dLLM on NVIDIA B200 (sm_100a).
 *
 * C ABI.  One non-block-entry denoising step of one layer is
 *     focus_select_queries  ->  [probe layer: focus_dense_attn (emits LSE) -> focus_find_sinks]
 *     ->  focus_score_blocks  ->  focus_select_blocks  ->  focus_sparse_attn
 *
 * Conventions shared by every entry point
 *   - Positions are 0-indexed: prompt [0, M), response / gen region [M, L).  Prompt block b is
 *     [b*kv_block, min((b+1)*kv_block, M)); there are nb = ceil(M / kv_block) blocks.
 *   - Query head h reads KV head g(h) = h / (n_q_heads / n_kv_heads).
 *   - All data pointers are DEVICE pointers owned by the caller unless a comment says "host".
 *     Tensor base pointers (Q, K, V, O, pooled keys, logits, new K/V rows) must be 16-byte aligned; the innermost
 *     (head_dim) dimension is contiguous; token and head strides are in elements and must be multiples of 8
 *     elements.  Both are checked on the host (FOCUS_ERR_INVALID_ARG): a misaligned address would fault on the device.
 *   - Index outputs are int32, ascending, padded with -1.  Counts are written to device int32 so a
 *     whole step can be enqueued without a host round trip.
 *   - Every call validates its arguments on the host, enqueues its kernels on the caller's stream and
 *     returns without synchronising.  Nothing is allocated after focus_create: scratch comes from the
 *     context's workspace (FOCUS_ERR_WORKSPACE_TOO_SMALL if it does not fit).  Calls on one context
 *     must be issued on one stream at a time (they share the workspace).
 *   - Stream order.  The attention kernels and the selection kernel of focus_sparse_layer are launched with
 *     programmatic stream serialization and let their successor in the stream begin early; each of them waits
 *     for its predecessor to complete before it writes anything, and before it reads anything that another of
 *     these kernels may have written (outputs, lists, workspace).  A kernel of another library placed after a call
 *     sees complete results.  Ahead of that wait these kernels read only inputs that none of them writes:
 *     focus_sparse_layer reads Q, the focus and sink index lists, the pooled keys and the sinks' K/V rows there,
 *     its attention kernel the row list and Q; focus_dense_attn and focus_sparse_attn read nothing ahead of it.
 *     Such an input is complete if its producer finished before the call's predecessor in the stream started, or if
 *     the producer is a kernel of this library (those make their outputs visible before they exit).  An input
 *     written by a foreign kernel that runs immediately before a focus_sparse_layer call, with nothing in between
 *     on the stream, would be read in the window between that kernel's last block exiting and its writes being
 *     guaranteed visible: put any other kernel or an event wait in between, or set FOCUS_OPT_NO_PDL.  And do not
 *     feed the O or lse of one attention call straight in as the Q, q_rows or n_rows of the next attention or
 *     focus_sparse_layer call with no other kernel in between: those three are read ahead of the wait.
 *   - Results are deterministic run to run (fixed reduction order, no floating-point atomics).
 *   - A device-side anomaly (index out of range, a bounded wait that ran out) never traps: the kernel
 *     skips the access, records a code in the context's device status word and returns; read it with
 *     focus_poll_status.
 *   - Every compute entry point opens an NVTX range of its own name around its launches (host side), so a profiler
 *     attached to the process can group kernels by stage.
 *   - There is no CPU fallback: without a CUDA device every compute entry point fails.
 */
#ifndef FOCUS_H_
#define FOCUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct focus_ctx focus_ctx;          /* opaque: device, SM count, workspace, status word */
typedef struct CUstream_st* focus_stream;    /* same type as cudaStream_t */

typedef enum {
  FOCUS_OK = 0,
  FOCUS_ERR_INVALID_ARG = 1,
  FOCUS_ERR_UNSUPPORTED = 2,
  FOCUS_ERR_WORKSPACE_TOO_SMALL = 3,
  FOCUS_ERR_CUDA = 4,
  FOCUS_ERR_TIMEOUT = 5
} focus_status;

typedef enum { FOCUS_F32 = 0, FOCUS_BF16 = 1 } focus_dtype;

/* How block scores are reduced over heads.  PER_KV_GROUP: one block set per KV head, scored by the
 * mean over the query heads of that group (for MHA: per head).  ALL: one block set for the layer,
 * scored by the mean over all heads (Eq. 7 as printed). */
typedef enum { FOCUS_HEADS_PER_KV_GROUP = 0, FOCUS_HEADS_ALL = 1 } focus_head_reduce;

/* How sink tokens join the key set.  TOKENS: as single tokens (Eq. 8 as printed).  BLOCKS: the prompt
 * block around each sink token is added to the block list. */
typedef enum { FOCUS_SINK_TOKENS = 0, FOCUS_SINK_BLOCKS = 1 } focus_sink_mode;

typedef struct {
  int32_t L, M;                    /* total positions, prompt length */
  int32_t n_q_heads, n_kv_heads;   /* H, Hkv; H % Hkv == 0 */
  int32_t head_dim;                /* 64 or 128 */
  int32_t kv_block;                /* prompt block size B: 64 or 128 */
  int32_t dtype;                   /* focus_dtype of Q, K, V and O */
  float softmax_scale;             /* 0 => 1/sqrt(head_dim) */
  int64_t q_stride_row, q_stride_head;    /* Q[(pos - q_base)*q_stride_row + h*q_stride_head + c] */
  int64_t kv_stride_tok, kv_stride_head;  /* K[g*kv_stride_head + j*kv_stride_tok + c], same for V */
} focus_shape;

/* ---- context ------------------------------------------------------------------------------- */

/* Creates a context on `device` and allocates its workspace (workspace_bytes == 0: 256 MiB) and a
 * 4-byte status word.  The only entry point that allocates.  Errors: INVALID_ARG (null out pointer),
 * CUDA (no such device / allocation failed). */
focus_status focus_create(focus_ctx** out, int device, size_t workspace_bytes);
focus_status focus_destroy(focus_ctx* ctx);

/* Upper bound of the scratch any single call needs for this shape with at most n_q query rows,
 * max_blocks blocks per group and n_sink sink tokens. */
focus_status focus_workspace_bytes(const focus_shape* shape, int32_t n_q, int32_t max_blocks, int32_t n_sink,
                                   size_t* out_bytes);

/* Synchronises `stream`, copies the device status word to *device_status (0 = clean, else the
 * focus_status code of the first anomaly) and clears it. */
focus_status focus_poll_status(focus_ctx* ctx, focus_stream stream, int32_t* device_status);
const char* focus_status_string(focus_status s);

/* Number of kernels this library has launched in this process so far (all contexts). */
uint64_t focus_launch_count(void);

/* Which attention kernel the last focus_dense_attn / focus_sparse_attn / focus_sparse_layer call on this context
 * used: 1 = generic SIMT, 2 = tensor-core kernel with one 128-row query tile per CTA, 3 = tensor-core kernel with
 * two query tiles per CTA (taken for >= 256 stacked rows per KV head and >= 24 key tiles per CTA), 4 = tensor-core
 * kernel with one query tile and two softmax warpgroups on alternating key tiles (>= 128 stacked rows per KV head
 * and >= 4 key tiles per CTA, where 3 does not apply); 0 = none yet. */
int32_t focus_last_attn_variant(focus_ctx* ctx);

/* Selects the attention implementation for bf16 inputs (head_dim 128 or 64): 0 = automatic (tensor-core
 * kernel where supported), 1 = force the generic SIMT kernels.  Returns the previous value. */
int32_t focus_set_force_simt(focus_ctx* ctx, int32_t force);

/* Launch options of the attention kernels (no counterpart in the paper): every one of them selects between
 * implementations that return the same results, for tests that must reach a fallback and for A/B measurements.
 *   FOCUS_OPT_MERGE_MODE  how the key splits of a query tile are merged: 0 = automatic (inside a thread-block cluster
 *                         where all clusters of the launch are resident), 1 = through global memory by the CTA that
 *                         arrives last at the tile's counter, 2 = through global memory by a separate kernel
 *   FOCUS_OPT_NO_WIDE     1 = never use the three-warpgroup kernels (variants 3 and 4 of focus_last_attn_variant)
 *   FOCUS_OPT_NO_PDL      1 = plain stream order, no programmatic dependent launches
 * Returns the previous value, or -1 for a bad context, option or value. */
typedef enum { FOCUS_OPT_MERGE_MODE = 0, FOCUS_OPT_NO_WIDE = 1, FOCUS_OPT_NO_PDL = 2 } focus_option;
int32_t focus_set_option(focus_ctx* ctx, int32_t option, int32_t value);

/* Self-test of the bounded waits (no counterpart in the paper).  Every wait on a barrier inside the tensor-core
 * kernels gives up after a time limit, records FOCUS_ERR_TIMEOUT in the status word and lets the kernel unwind
 * instead of spinning for ever.  This call launches one small CTA that waits, with a limit of limit_us microseconds
 * (1 .. 100 000), on a barrier nobody ever arrives at: afterwards focus_poll_status must report
 * FOCUS_ERR_TIMEOUT and the context must still be usable.  Nothing else is touched.  Errors: INVALID_ARG. */
focus_status focus_selftest_bounded_wait(focus_ctx* ctx, int32_t limit_us, focus_stream stream);

/* Measurement aid (no counterpart in the paper): streams the `bytes` bytes at device pointer `ptr` once, read only,
 * with 128-bit loads from every SM, and leaves the 32-bit xor of all 32-bit words read in *checksum (device memory,
 * overwritten).  Its bandwidth is the practical HBM read ceiling on the device at hand, which the figures of the
 * HBM-bound kernels are put beside.  ptr must be 16-byte aligned and bytes a multiple of 16 (0 is allowed: checksum
 * 0).  One memset and one launch on `stream`; the buffer stays the caller's.  Errors: INVALID_ARG, CUDA. */
focus_status focus_stream_read(focus_ctx* ctx, const void* ptr, size_t bytes, uint32_t* checksum, focus_stream stream);

/* ---- stage 1: past-confidence indicator (Eq. 4) and window expansion (Eq. 5) ---------------- */

/* I_focus = the k positions i in [blk_lo, blk_hi) with masked[i] != 0 that have the highest
 * conf_prev[i] (ties: lower index; NaN ranks last); n_focus = min(k, number of candidates).
 * I_active = union over i in I_focus of [i - w/2, i + w/2] (integer division) clipped to
 * [clip_lo, clip_hi).
 *   conf_prev  float[L], masked uint8[L]
 *   focus_idx  int32[k]; active_idx int32[k * (2*(w/2) + 1)]; n_focus, n_active int32[1]
 * Requires 0 <= blk_lo <= blk_hi <= L, blk_hi - blk_lo <= 4096, 0 <= k <= 1024, w >= 0. */
focus_status focus_select_queries(focus_ctx* ctx, const float* conf_prev, const uint8_t* masked, int32_t L,
                                  int32_t blk_lo, int32_t blk_hi, int32_t k, int32_t w,
                                  int32_t clip_lo, int32_t clip_hi,
                                  int32_t* focus_idx, int32_t* n_focus,
                                  int32_t* active_idx, int32_t* n_active, focus_stream stream);

/* ---- stage 2: attention-sink identification (Eq. 6) ----------------------------------------- */

/* S_j = mean over heads h and active rows i of softmax_j(scale * q_i^h . k_j^{g(h)}), the softmax
 * taken over all L keys; I_sink = the n_sink positions of [cand_lo, cand_hi) with the highest S_j
 * (ties: lower index).
 *   Q          rows for positions [q_base, ...): the row of position p starts at (p - q_base)*q_stride_row
 *   active_idx int32[max_active] positions (from focus_select_queries), n_active int32[1] on device
 *   K          [Hkv, L, d] by strides
 *   lse        float[H * max_active] (lse[h*max_active + r], natural log, as written by focus_dense_attn
 *              for the same rows) or NULL: the library then computes it (one more pass over K)
 *   sink_idx   int32[n_sink] (may be NULL when n_sink == 0: scores only); scores float[L] or NULL (receives S)
 * n_active == 0 on the device is recorded as INVALID_ARG in the status word (outputs are -1). */
focus_status focus_find_sinks(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                              const int32_t* active_idx, const int32_t* n_active, int32_t max_active,
                              const void* K, const float* lse, int32_t n_sink,
                              int32_t cand_lo, int32_t cand_hi,
                              int32_t* sink_idx, float* scores, focus_stream stream);

/* The Top-N_sink step of Eq. 6 on its own: I_sink = the n_sink positions of [cand_lo, cand_hi) with the highest
 * scores[j] (ties: lower index), ascending, padded with -1 when the range is shorter than n_sink.  For a layer whose
 * heads live on several devices (equal head counts): each device computes S over its own heads with
 * focus_find_sinks (n_sink = 0, sink_idx NULL, scores = its S), the S are averaged over the devices -- L floats, the
 * only exchange of a denoising step -- and every device selects from the average with this call.
 *   scores float[L], sink_idx int32[n_sink] (device) */
focus_status focus_select_sinks(focus_ctx* ctx, const float* scores, int32_t L, int32_t cand_lo, int32_t cand_hi,
                                int32_t n_sink, int32_t* sink_idx, focus_stream stream);

/* ---- stage 3: block relevance (Eq. 7) and Top-C selection (Eq. 8) --------------------------- */

/* K-bar[g, b, :] = mean of the keys of prompt block b (float[Hkv * nb * d]); run once per KV-cache
 * refresh so that focus_score_blocks need not stream K again. */
focus_status focus_pool_keys(focus_ctx* ctx, const focus_shape* shape, const void* K, float* Kbar,
                             focus_stream stream);

/* R[g, b] = mean over the focus rows i and the heads h of group g of q_i^h . K-bar_b^{g(h)} (no
 * softmax, no 1/sqrt(d)); G = Hkv rows (PER_KV_GROUP) or one row holding the mean over all heads (ALL).
 * Exactly one of K (pooled on the fly, one pass over the prompt keys) and Kbar (from
 * focus_pool_keys) must be non-NULL.  focus_idx int32[max_focus], n_focus int32[1] on device.
 * R float[G * nb]. */
focus_status focus_score_blocks(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base,
                                const int32_t* focus_idx, const int32_t* n_focus, int32_t max_focus,
                                const void* K, const float* Kbar, int32_t head_reduce,
                                float* R, focus_stream stream);

/* focus_score_blocks for callers that cannot allocate device memory.  (The paper has no counterpart: this is a
 * deployment variant of the Eq. 7 scorer above, computing the same R.)
 *
 * Who needs it: code that runs inside another component's memory budget (a serving process whose pool already
 * owns the GPU), code for which cudaMalloc's implicit synchronisation is off limits, or a plug-in that is given a
 * stream and buffers and nothing else.  Such callers cannot call focus_create, which allocates the workspace, so
 * this entry point takes no context, and it calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Its scratch (the mean focus query per KV head; in FOCUS_HEADS_ALL mode also the per-group scores) is a fixed
 * 288.25 KiB array inside the library that every GPU loading the library holds until the process exits.  Limits,
 * rejected with FOCUS_ERR_WORKSPACE_TOO_SMALL before anything is launched: n_kv_heads * head_dim <= 8192 and, in
 * FOCUS_HEADS_ALL mode, n_kv_heads * nb <= 65536.
 *
 * The first call on each device looks up the array's device address (that device must be current); if nothing of
 * the library has run on that device yet, this lookup is also the moment the runtime loads the library's device
 * code there and places the array.  Make that first call before any stream capture begins.  All calls share the one array and it keeps the previous call's
 * contents; every element a call reads it has first rewritten, so nothing needs clearing, but two calls whose
 * kernels overlap on the GPU (different streams, or several processes' worth of threads on one context) race on
 * it: serialise them.
 *
 * Arguments as focus_score_blocks, minus the context; device_status (device int32, caller-owned) receives the
 * code of a device-side anomaly (bad focus index, empty focus set) or may be NULL. */
focus_status focus_score_blocks_static(const focus_shape* shape, const void* Q, int32_t q_base,
                                       const int32_t* focus_idx, const int32_t* n_focus, int32_t max_focus,
                                       const void* K, const float* Kbar, int32_t head_reduce,
                                       float* R, int32_t* device_status, focus_stream stream);

/* Per row g of R: the C highest-scoring blocks (ties: lower index), ascending, into
 * block_idx[g*max_blocks ...] (padded -1), count into block_cnt[g].
 * SINK_TOKENS: sink_keep[g*n_sink + s] = 1 iff sink token s lies outside every selected block of g.
 * SINK_BLOCKS: the blocks containing the sink tokens are merged into the list (sink_keep all 0);
 *              needs max_blocks >= min(nb, C + n_sink).
 * Requires 0 <= C <= nb, max_blocks >= C, nb <= 8192.  sink_idx int32[n_sink] on device. */
focus_status focus_select_blocks(focus_ctx* ctx, const focus_shape* shape, const float* R, int32_t head_reduce,
                                 int32_t C, const int32_t* sink_idx, int32_t n_sink, int32_t sink_mode,
                                 int32_t* block_idx, int32_t max_blocks, int32_t* block_cnt,
                                 uint8_t* sink_keep, focus_stream stream);

/* ---- stage 4: sparse attention (Eq. 9) and the dense attention of the dense layers ---------- */

/* o_i^h = sum_{j in keys(h)} softmax_j(scale * q_i^h . k_j) v_j with keys(h) = tokens of the selected
 * blocks of the head's group + kept sink tokens + every response position [M, L), each counted once.
 *   Q        rows for positions [q_base, q_base + n_q)
 *   q_rows   int32[max_rows] positions to compute (device) with n_rows int32[1] (device), or both NULL:
 *            all n_q rows (then max_rows is ignored)
 *   block_idx/block_cnt/sink_idx/sink_keep as written by focus_select_blocks (head_reduce tells whether
 *            there is one list per KV head or one shared list); sink_keep may be NULL when n_sink == 0
 *   O        [rows, H, d] contiguous, input dtype; output row r belongs to q_rows[r]
 *   lse      float[H * rows_bound] (lse[h*rows_bound + r], rows_bound = max_rows or n_q) or NULL */
focus_status focus_sparse_attn(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base, int32_t n_q,
                               const int32_t* q_rows, const int32_t* n_rows, int32_t max_rows,
                               const void* K, const void* V, int32_t head_reduce,
                               const int32_t* block_idx, int32_t max_blocks, const int32_t* block_cnt,
                               const int32_t* sink_idx, const uint8_t* sink_keep, int32_t n_sink,
                               void* O, float* lse, focus_stream stream);

/* One whole sparse layer (Algorithm 1, sparse branch) in one call, for the default modes (one block set per
 * KV head, sinks as tokens) with cached pooled keys: block relevance (Eq. 7) -> Top-C (Eq. 8) -> sparse
 * attention (Eq. 9).  Same results as focus_score_blocks(Kbar) + focus_select_blocks + focus_sparse_attn with
 * max_blocks = C, in fewer kernel launches.  Outputs: R float[Hkv*nb] (required unless the tensor-core path is
 * taken; may then be NULL), block_idx int32[Hkv*C], block_cnt int32[Hkv], sink_keep uint8[Hkv*n_sink], O, lse. */
focus_status focus_sparse_layer(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base, int32_t n_q,
                                const int32_t* q_rows, const int32_t* n_rows, int32_t max_rows,
                                const int32_t* focus_idx, const int32_t* n_focus, int32_t max_focus,
                                const void* K, const void* V, const float* Kbar, int32_t C,
                                const int32_t* sink_idx, int32_t n_sink, float* R, int32_t* block_idx,
                                int32_t* block_cnt, uint8_t* sink_keep, void* O, float* lse, focus_stream stream);

/* Bidirectional softmax attention of the same rows over all L keys ("FullAttn" of Algorithm 1): the
 * dense layers, the probe layer (its lse feeds focus_find_sinks) and the baseline of the benchmark. */
focus_status focus_dense_attn(focus_ctx* ctx, const focus_shape* shape, const void* Q, int32_t q_base, int32_t n_q,
                              const int32_t* q_rows, const int32_t* n_rows, int32_t max_rows,
                              const void* K, const void* V, void* O, float* lse, focus_stream stream);

/* ---- closing the decoding loop around the attention path ------------------------------------------ */

/* Eq. 2: for each listed position, the predicted token argmax_v p(v) (lowest v on ties; NaN logits count as
 * -inf) and its confidence c = max_v p(v), p = softmax over the vocabulary of that position's logits row.
 * The confidences are the conf_prev of the next step's focus_select_queries; the same selection call with
 * k = n^(t) and w = 0 picks the positions to unmask (the unmasking rule of the section on diffusion LLM inference).
 *   logits    [n_pos rows, vocab] for positions [pos_base, pos_base + n_pos), dtype FOCUS_F32 or FOCUS_BF16;
 *             row_stride in elements, a multiple of 8 (bf16) / 4 (f32); base 16-byte aligned
 *   rows      int32[max_rows] positions (device) with n_rows int32[1] (device), or both NULL: the first max_rows
 *             positions
 *   conf      float[max_rows], token int32[max_rows]; entries beyond n_rows are 0 and -1. */
focus_status focus_confidence(focus_ctx* ctx, const void* logits, int32_t dtype, int64_t row_stride, int32_t vocab,
                              int32_t pos_base, int32_t n_pos, const int32_t* rows, const int32_t* n_rows,
                              int32_t max_rows, float* conf, int32_t* token, focus_stream stream);

/* Eq. 3; Algorithm 1, the cache-update step of the non-block-entry branch: the key and value states computed this
 * step for the listed positions replace the cached rows; every other row keeps its cached state.
 *   K_cache, V_cache  [Hkv, L, d] by the shape's strides (updated in place)
 *   K_new, V_new      [max_rows, Hkv, d] contiguous; row r belongs to position rows[r]
 *   rows int32[max_rows], n_rows int32[1] (device).  Positions outside [0, L) are skipped and reported through
 * the status word.  Pooled keys are not touched: the listed positions of a non-block-entry step lie in the
 * response region; after a block-entry refresh of prompt rows call focus_pool_keys again. */
focus_status focus_update_kv(focus_ctx* ctx, const focus_shape* shape, void* K_cache, void* V_cache,
                             const void* K_new, const void* V_new, const int32_t* rows, const int32_t* n_rows,
                             int32_t max_rows, focus_stream stream);

/* Incremental maintenance of the pooled keys after focus_update_kv (Eq. 3 applied to prompt rows, e.g. at a
 * block-entry refresh; K-bar_b of "Block-wise token pruning"): K-bar[g, b, :] is recomputed for exactly the prompt
 * blocks b that hold one of the listed positions, from the (already refreshed) K cache, with the arithmetic of
 * focus_pool_keys -- the result equals a full focus_pool_keys of the refreshed cache bit for bit.  Listed positions in
 * the response region change no pooled key.  rows int32[max_rows] ascending (device), n_rows int32[1] (device).
 * Negative positions are skipped and reported through the status word. */
focus_status focus_update_pooled_keys(focus_ctx* ctx, const focus_shape* shape, const void* K, float* Kbar,
                                      const int32_t* rows, const int32_t* n_rows, int32_t max_rows,
                                      focus_stream stream);

/* The state update that ends a denoising step (Algorithm 1, last line of the step loop; the unmasking rule stated
 * after Eq. 2), on the device, so that a multi-step loop needs no host-side mask handling.
 *   conf_new, token_new  float / int32 [max_rows] as written by focus_confidence for the rows evaluated this step;
 *                        the row list (rows, n_rows, max_rows; or NULL, NULL: positions pos_base .. pos_base+max_rows-1)
 *                        is the one given to focus_confidence and must be ascending
 *   conf    float[L]   c^(t) -> c^(t+1): conf[pos] = conf_new[r] for every evaluated position (others keep their value)
 *   masked  uint8[L], x int32[L] (token ids): among the evaluated positions that are still masked and lie in the
 *           decoding block [blk_lo, blk_hi), the n_unmask with the highest new confidence (ties: lower position; NaN
 *           last; fewer if there are fewer candidates) get x[pos] = token_new[r] and masked[pos] = 0; every other
 *           position stays as it is (the rest remains masked)
 *   unmasked_idx int32[n_unmask] receives those positions ascending, padded with -1 (may be NULL when n_unmask == 0);
 *           n_unmasked int32[1] their count (may be NULL)
 * Requires max_rows <= 4096 and n_unmask <= 4096.  One launch.  Positions outside [0, L) are skipped and reported
 * through the status word. */
focus_status focus_commit_step(focus_ctx* ctx, const float* conf_new, const int32_t* token_new, int32_t pos_base,
                               const int32_t* rows, const int32_t* n_rows, int32_t max_rows, int32_t L,
                               int32_t blk_lo, int32_t blk_hi, int32_t n_unmask, float* conf, uint8_t* masked,
                               int32_t* x, int32_t* unmasked_idx, int32_t* n_unmasked, focus_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* FOCUS_H_ */

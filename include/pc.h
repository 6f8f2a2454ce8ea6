/*
 * libpc: the attention hot path of ParallelComp (arXiv 2502.14317, Sec. 3.1) for one
 * layer on one B200 (sm_100a).  C ABI, plain pointers and sizes.
 *
 * Notation.  A long input is cut into C chunks; every chunk is followed by the same
 * query window of w tokens, so a chunk holds L = ctx + w tokens, with RoPE positions
 * 0..L-1 restarting in every chunk (position reuse).  Hq query heads, Hkv key/value
 * heads, G = Hq / Hkv, head size d.  m chunks and k tokens per (kept chunk, kv-head)
 * survive eviction; the compressed cache has Nk = m * k entries per kv-head.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers, 16-byte aligned, bf16 unless stated
 *     otherwise; d is the contiguous dimension; strides are in elements and must be
 *     multiples of 8.  Descriptor structs and stride arrays are HOST memory.
 *   - The caller owns every buffer.  The library allocates no device memory and keeps
 *     no state between calls (pc_parallel_attn_static, below, is the one exception: its
 *     scratch is an array inside the library image); scratch comes from the caller's
 *     workspace, sized by the matching *_workspace_bytes query (host function, no GPU work).
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and return without synchronising.  Index outputs of one call
 *     are device inputs of the next, so the five calls chain on one stream with no
 *     host round trip.
 *   - Return value: PC_OK or a negative pc_status.  Argument errors are found on the
 *     host before anything is launched; nothing is written in that case.
 *   - `status_word` (device int32, may be NULL) is left untouched on success; a kernel
 *     whose bounded wait on a copy or tensor-core barrier ran out stores a positive code
 *     naming that wait there (the condition PC_ERR_TIMEOUT stands for) and the results of
 *     that call are undefined.  The caller clears it and
 *     reads it after synchronising.  No kernel spins without a limit.
 *   - Supported: d in {64, 128}; Hq % Hkv == 0; any window 1 <= w < L with w <= 128;
 *     G * w <= 1024 (the window rows of all G heads of a kv-head are swept in passes of up to 256 rows).
 */
#ifndef PC_H_
#define PC_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define PC_API __attribute__((visibility("default")))
#else
#define PC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PC_OK = 0,
  PC_ERR_INVALID_ARG = -1,   /* null pointer, bad size, misaligned pointer or stride      */
  PC_ERR_UNSUPPORTED = -2,   /* shape outside the supported set, or device is not sm_100  */
  PC_ERR_WORKSPACE = -3,     /* workspace missing or smaller than *_workspace_bytes       */
  PC_ERR_CUDA = -4,          /* a CUDA runtime / driver call failed                       */
  PC_ERR_TIMEOUT = -5,       /* value stored in status_word by a kernel whose wait ran out */
  PC_ERR_SCRATCH_LIMIT = -6  /* pc_parallel_attn_static: the shape needs more than PC_STATIC_SCRATCH_BYTES */
} pc_status;

/* Text for a status code (static storage). */
PC_API const char* pc_status_string(int32_t status);

/* Library version, major * 1000 + minor. */
PC_API int32_t pc_version(void);

/* Number of kernels the library has launched in this process so far (all calls, all streams, all devices):
 * the difference of two readings counts the launches in between.  Host-side counter, no GPU work. */
PC_API uint64_t pc_launch_count(void);

/* ------------------------------------------------------------------------------------
 * Chunk-local causal attention with position reuse and fused query-window scores.
 * Paper: Sec. 3.1 "Parallel attention" (chunking, Eq. 1-2) and "Parallel KV cache
 * eviction" (Eq. 5-6).
 *
 * For every chunk c and q-head h (kv-head h / G), with q', k' = RoPE(q), RoPE(k) at the
 * token's chunk-local position (pairs (t, t + d/2), angle p * theta^(-2t/d)) rounded to
 * bf16:
 *     A = softmax(q' k'^T * scale + causal mask),  O = A v                      (Eq. 1-2)
 *     win_score[c, hkv, j] = sum_{g < G} sum_{i = L-w}^{L-1} A[c, hkv*G+g, i, j]    (Eq. 6)
 * The score is accumulated inside the attention kernel (second sweep of the window rows
 * against the final log-sum-exp); it is not a separate launch.
 *
 * q [C,L,Hq,d], k, v [C,L,Hkv,d]: inputs before RoPE, addressed through the element
 * strides (chunk, token, head) in the descriptor.  Queries and keys are rotated by a pass
 * of their own ahead of the attention kernel (the rotated queries live in the workspace).
 * chunk_len [C] int32 (device; NULL: every chunk holds L tokens): tokens of chunk c, window
 * included - the paper cuts the input into chunks of AT MOST the trained length.  The
 * window of a shorter chunk directly follows its context (positions len-w .. len-1); keys
 * at or behind len are masked; o, lse and win_score read as zero at positions >= len.
 * Values outside (w, L] are clamped into that range.  The rows of k and v behind len must
 * hold finite numbers (they meet zero probabilities).  pc_select_tokens then ranks such a
 * chunk with n_cand = len - w (a call of its own for that chunk).
 * o [C,L,Hq,d] (strides o_stride), k_rot [C,L,Hkv,d] contiguous (rotated keys, what the
 * gather later copies; may be NULL, then it lives in the workspace), lse [C,Hq,L] fp32
 * natural-log log-sum-exp of every row (may be NULL), win_score [C,Hkv,L] fp32,
 * win_lse [C,Hq,w] fp32 (rows len-w..len-1 of each chunk).
 * Workspace: pc_chunk_prefill_attn_workspace_bytes(desc) - cos/sin tables and the rotated
 * queries (C*L*Hq*d bf16) - plus, if k_rot is NULL, C*L*Hkv*d*2 bytes rounded up to a
 * multiple of 256 for the rotated keys.
 */
typedef struct {
  int32_t C, L, w, Hq, Hkv, d;
  float rope_theta;
  float softmax_scale;                 /* 0 -> 1/sqrt(d) */
  int64_t q_stride[3], k_stride[3], v_stride[3], o_stride[3];   /* chunk, token, head; 0,0,0 -> contiguous */
} pc_prefill_desc;

PC_API size_t pc_chunk_prefill_attn_workspace_bytes(const pc_prefill_desc* desc);

PC_API int32_t pc_chunk_prefill_attn(const pc_prefill_desc* desc, const void* q, const void* k, const void* v,
                              const int32_t* chunk_len, void* o, void* k_rot, float* lse, float* win_score,
                              float* win_lse, int32_t* status_word, void* workspace, size_t workspace_bytes,
                              void* stream);

/* ------------------------------------------------------------------------------------
 * Test hook for the bounded device-side waits (no counterpart in the paper).
 * Every wait of a kernel on a copy or tensor-core barrier gives up after a limit, stores a
 * positive code naming the wait in the call's status_word, lets the kernel drain what is in
 * flight and return; the host then treats the call's results as undefined (PC_ERR_TIMEOUT).
 *   wait_limit_cycles      limit for all later launches of this process (0: the default of
 *                          about 2e9 cycles, a second);
 *   skip_final_publication non-zero: the single-CTA chunk-prefill kernel (head size 64, or an
 *                          odd number of q-heads per kv-head) leaves out ONE signal that carries
 *                          no data - the "no more work" message to its consumer warps after the
 *                          last work item, when nothing is in flight any more - so that their
 *                          wait runs out.  Outputs of such a call are complete; its status_word
 *                          is non-zero.  Zero switches the hook off again.
 * Host-side settings, read at every launch.
 */
PC_API int32_t pc_debug_bounded_wait_test(int64_t wait_limit_cycles, int32_t skip_final_publication);

/* ------------------------------------------------------------------------------------
 * RoPE with position reuse on its own.  Paper: Sec. 3.1 "Parallel attention" (the position
 * encodings of every chunk restart at 0).
 *     y[c, p, h, :] = bf16( RoPE(x[c, p, h, :]) at position p ),  pairs (t, t + d/2),
 *     angle p * theta^(-2t/d), evaluated so that the result equals the fp64 rotation
 *     rounded once to bf16.
 * This is the pass pc_chunk_prefill_attn runs over its queries and keys before the attention
 * kernel (same kernel), offered for callers that want rotated queries or keys as tensors.  x, y [C,L,H,d] bf16 contiguous.
 * Workspace: pc_rope_position_reuse_workspace_bytes(L, d) (cos/sin tables).
 */
PC_API size_t pc_rope_position_reuse_workspace_bytes(int32_t L, int32_t d);

PC_API int32_t pc_rope_position_reuse(const void* x, int32_t C, int32_t L, int32_t H, int32_t d, float rope_theta,
                                void* y, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * Stand-in for the chunk self-information I_c of Eq. 3 in a single-layer setting
 * (the true I_c = -log P(X^q | X^c) needs the whole model; it enters pc_select_chunks
 * as an input array).  chunk_score[c] = - mean over q-heads and window rows of
 * win_lse[c, h, i].  Not part of the paper; used by the synthetic pipeline only.
 * win_lse [C,Hq,w] fp32 -> chunk_score [C] fp32.
 */
PC_API int32_t pc_chunk_score_from_lse(const float* win_lse, int32_t C, int32_t Hq, int32_t w, float* chunk_score,
                                void* stream);

/* ------------------------------------------------------------------------------------
 * Chunk eviction.  Paper: Sec. 3.1 "Chunk eviction", Eq. 3-4 (fixed-size queue keeping
 * the chunks with the lowest self-information).
 * Keeps the m best of C scores (lowest if lower_is_better != 0); ties go to the lower
 * chunk id; NaN ranks worst; kept[m] lists the chunk ids in ascending order.
 * 1 <= m <= C <= 1024.
 */
PC_API int32_t pc_select_chunks(const float* chunk_score, int32_t C, int32_t m, int32_t lower_is_better,
                         int32_t* kept, void* stream);

/* ------------------------------------------------------------------------------------
 * pc_chunk_score_from_lse followed by pc_select_chunks (same results, bit for bit) as one
 * call: for up to 64 chunks a single launch, which matters where the whole ranking stage
 * moves a few megabytes and is bound by launch latency.  Used by the synthetic single-layer
 * pipeline only (the stand-in score is not part of the paper).
 */
PC_API int32_t pc_score_select_chunks(const float* win_lse, int32_t C, int32_t Hq, int32_t w, int32_t m,
                                int32_t lower_is_better, float* chunk_score, int32_t* kept, void* stream);

/* ------------------------------------------------------------------------------------
 * Token eviction per kept chunk and kv-head.  Paper: Sec. 3.1 "Parallel KV cache
 * eviction", Eq. 7.
 * For row (r, hkv), r < m: the k largest of win_score[kept[r], hkv, 0..n_cand) (window
 * keys j >= n_cand are never candidates); ties go to the lower position; NaN ranks
 * worst; -0 == +0.  idx[m,Hkv,k] int32 holds the positions in ascending order; if
 * k > n_cand the tail is filled with -1.  `kept` is a device array (output of
 * pc_select_chunks).  n_cand <= L, n_cand <= 32768.
 */
PC_API int32_t pc_select_tokens(const float* win_score, const int32_t* kept, int32_t C, int32_t m, int32_t Hkv,
                         int32_t L, int32_t n_cand, int32_t k, int32_t* idx, void* stream);

/* ------------------------------------------------------------------------------------
 * Token eviction with attention calibration.  Paper: Sec. 3.1 "Attention calibration", Eq. 8,
 * with the regions of App. C; combined here with the top-k of Eq. 7.
 * For row (r, hkv): first evict every candidate j < n_cand whose score
 * win_score[kept[r], hkv, j] EXCEEDS the threshold of its region - lambda_s for the first n_s
 * positions (sink tokens, R_s), lambda_r for the last n_r candidate positions (recency
 * tokens, R_r), lambda_m for the rest (R_m); +infinity switches a region off - then keep the
 * k largest of the survivors as pc_select_tokens does (ties to the lower position, NaN is
 * never above a threshold and ranks worst, ascending output).  Where fewer than k survive,
 * the tail of idx[r,hkv,:] is -1 (pc_gather_kv turns those into zero rows).  The comparison
 * is made on the fp32 score against the fp32 threshold.  Same limits as pc_select_tokens;
 * n_s, n_r >= 0; where the first two regions overlap the sink region wins.
 */
PC_API int32_t pc_select_tokens_calibrated(const float* win_score, const int32_t* kept, int32_t C, int32_t m,
                                    int32_t Hkv, int32_t L, int32_t n_cand, int32_t k, int32_t n_s, int32_t n_r,
                                    float lambda_s, float lambda_m, float lambda_r, int32_t* idx, void* stream);

/* ------------------------------------------------------------------------------------
 * Compressed cache.  Paper: Eq. 7 (K[R], V[R]) and Eq. 9 (concatenation over chunks).
 *     k_out[hkv, r*k + t, :] = k_src[kept[r], idx[r,hkv,t], hkv, :]     (same for v)
 *     pos_out[hkv, r*k + t]  = idx[r,hkv,t]
 * k_src (rotated keys) and v_src are [C,L,Hkv,d] addressed by kv_stride (element strides of
 * chunk, token, head; host array of 3; [L*Hkv*d, Hkv*d, d] for contiguous tensors); outputs are contiguous [Hkv, m*k, d] and
 * [Hkv, m*k] int32 (pos_out may be NULL).  Entries with idx < 0 give zero rows and
 * position -1.  Pure bit copy.
 */
PC_API int32_t pc_gather_kv(const void* k_src, const void* v_src, const int64_t* kv_stride, const int32_t* kept,
                     const int32_t* idx, int32_t m, int32_t Hkv, int32_t k, int32_t d,
                     void* k_out, void* v_out, int32_t* pos_out, void* stream);

/* ------------------------------------------------------------------------------------
 * Online chunk queue.  Paper: Sec. 3.1 "Chunk eviction" (the kept chunks live in a priority
 * queue of fixed size so that prefilling stays inside the memory limit) together with
 * "Parallel KV cache eviction" applied to every chunk as it is produced (Sec. 5.5
 * "Throughput analysis": more chunks fit because only compressed caches persist).
 *
 * The chunks of a long input arrive in batches.  For every batch the caller runs
 * pc_chunk_prefill_attn, scores the chunks, runs pc_select_tokens over ALL chunks of the
 * batch (kept = 0..Cb-1) - or leaves that to pc_queue_select_gather below - then
 *   pc_queue_update  decides which of the m queued chunks and Cb new chunks stay: the m best
 *                    scores (lowest if lower_is_better != 0; ties go to the lower chunk id;
 *                    NaN ranks worst; empty slots rank below everything).  A chunk that stays
 *                    keeps its slot.  slot_src[s] = index within the batch of the chunk that
 *                    takes over slot s, or -1 where slot s keeps its contents.
 *   pc_queue_gather  copies the compressed cache of the chunks that moved in:
 *                        q_k[hkv, s*k + t, :] = k_src[c, idx[c,hkv,t], hkv, :],  c = slot_src[s] >= 0
 *                    (same for q_v; q_pos[hkv, s*k + t] = idx[c,hkv,t]); other slots are not touched.
 *                    After it the batch's full K/V may be overwritten by the next batch.
 * After the last batch pc_queue_emit lists the surviving chunk ids in ascending order in
 * kept_out[m] (slot_order[m] = their slots) and writes the compressed cache in that order,
 *     k_out[hkv, i*k + t, :] = q_k[hkv, slot_order[i]*k + t, :]   (same for v_out, pos_out),
 * which is bit for bit what pc_select_chunks + pc_select_tokens + pc_gather_kv give on all
 * chunks at once.  If fewer than m chunks were ever pushed the tail of kept_out and
 * slot_order is -1 and the corresponding rows are zero with position -1.
 *
 * State, owned by the caller and living on the device: q_score[m] fp32, q_chunk[m] int32
 * (chunk id, -1 = empty; set by pc_queue_init), q_k and q_v [Hkv, m*k, d] bf16,
 * q_pos [Hkv, m*k] int32.  chunk_score[Cb] is a device array; chunk ids of a batch are
 * chunk_id0 .. chunk_id0 + Cb - 1 and must be unique over the stream.  k_src, v_src, idx,
 * kv_stride as in pc_gather_kv with idx of shape [Cb,Hkv,k].  Limits: m + Cb <= 1024,
 * d in {64, 128}, 16-byte aligned K/V pointers.  Everything is enqueued on `stream`.
 */
PC_API int32_t pc_queue_init(int32_t m, float* q_score, int32_t* q_chunk, void* stream);

PC_API int32_t pc_queue_update(const float* chunk_score, int32_t Cb, int32_t chunk_id0, int32_t lower_is_better,
                        int32_t m, float* q_score, int32_t* q_chunk, int32_t* slot_src, void* stream);

PC_API int32_t pc_queue_gather(const void* k_src, const void* v_src, const int64_t* kv_stride,
                        const int32_t* slot_src, const int32_t* idx, int32_t m, int32_t Hkv, int32_t k, int32_t d,
                        void* q_k, void* q_v, int32_t* q_pos, void* stream);

/* pc_select_tokens and pc_queue_gather in one launch, for the chunks that enter the queue only (a chunk
 * that does not enter is dropped whole, so its tokens need no ranking): for every slot s with
 * c = slot_src[s] >= 0 and every kv-head, the k best of win_score[c, hkv, 0..n_cand) are ranked as
 * pc_select_tokens ranks them, their positions go to q_pos[hkv, s*k + t] and their rows of k_src / v_src
 * to q_k / q_v[hkv, s*k + t, :]; the block that ranked a row copies it, the index list never travels
 * through global memory.  Same results as the two calls.  win_score [Cb,Hkv,L] of the batch.
 * PC_ERR_UNSUPPORTED if k > 10240 (use the two calls then).
 */
PC_API int32_t pc_queue_select_gather(const float* win_score, const void* k_src, const void* v_src,
                               const int64_t* kv_stride, const int32_t* slot_src, int32_t m, int32_t Hkv,
                               int32_t L, int32_t n_cand, int32_t k, int32_t d, void* q_k, void* q_v,
                               int32_t* q_pos, void* stream);

PC_API int32_t pc_queue_emit(const int32_t* q_chunk, int32_t m, int32_t Hkv, int32_t k, int32_t d, const void* q_k,
                      const void* q_v, const int32_t* q_pos, int32_t* kept_out, int32_t* slot_order, void* k_out,
                      void* v_out, int32_t* pos_out, void* stream);

/* ------------------------------------------------------------------------------------
 * Parallel (global) attention of the query window over the compressed multi-chunk
 * cache.  Paper: Sec. 3.1 "Global attention", Eq. 9-11.
 * For each of B sequences: the w window queries (rotated here at positions
 * q_pos0..q_pos0+w-1, rounded to bf16) attend to all Nk cache entries of their kv-head
 * (every kept key precedes the window, so no mask) and causally to the window's own w
 * keys.  Keys arrive already rotated; the queries are rotated into the workspace first
 * (B * w * Hq * d * 2 bytes of it).  Small batches are split over key ranges with an fp32
 * merge; head size 128 with G * w a multiple of 256 and enough (sequence, kv-head) groups to fill the
 * GPU runs unsplit, one 256-row group per CTA pair.
 * q_win [B,w,Hq,d]; k_cache, v_cache [B,Hkv,Nk,d]; k_win, v_win [B,w,Hkv,d];
 * out [B,w,Hq,d] bf16; lse_out [B,Hq,w] fp32 natural log (may be NULL).  All contiguous.
 * Here w may be any power of two in [1, 128]: w = 1 is a decoding step over the compressed
 * cache (the paper keeps the cache for generation; the new token's own key/value are k_win,
 * v_win and the caller appends them to the cache afterwards).
 */
PC_API size_t pc_parallel_attn_workspace_bytes(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk);

PC_API int32_t pc_parallel_attn(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk,
                         const void* q_win, int32_t q_pos0, float rope_theta, float softmax_scale,
                         const void* k_cache, const void* v_cache, const void* k_win, const void* v_win,
                         void* out, float* lse_out, int32_t* status_word, void* workspace,
                         size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * Generation over the compressed cache (paper: Sec. 3.1 "Global attention" - the compressed
 * cache is what the following generation attends over; Table 7, per-token column).
 * pc_parallel_attn for caches stored with room to grow, followed by the append of the new
 * entries: k_cache, v_cache [B,Hkv,Nk_cap,d], of which the first Nk entries of every
 * (sequence, kv-head) are valid; the w new tokens (w = 1: one decoding step) attend to them
 * and causally to themselves exactly as in pc_parallel_attn, and afterwards, on the same
 * stream, their rotated keys and values k_win, v_win [B,w,Hkv,d] are copied to entries
 * Nk..Nk+w-1, so that the next step calls with Nk + w and q_pos0 + w.  Entries from Nk on are
 * never read by the attention.  PC_ERR_INVALID_ARG if Nk + w > Nk_cap.  Workspace:
 * pc_parallel_attn_workspace_bytes(B, w, Hq, Hkv, d, Nk).  Everything else as pc_parallel_attn.
 */
PC_API int32_t pc_parallel_attn_append(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk,
                                int32_t Nk_cap, const void* q_win, int32_t q_pos0, float rope_theta,
                                float softmax_scale, void* k_cache, void* v_cache, const void* k_win,
                                const void* v_win, void* out, float* lse_out, int32_t* status_word,
                                void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * pc_parallel_attn without a workspace argument, for callers that must not allocate.
 * The paper has no counterpart of this call: it computes exactly what pc_parallel_attn
 * computes (same kernels, same split plan, same results) and exists for the callers
 * below.
 *
 * Who needs it: code that runs where device allocation is off limits at call time -
 * an inference server that sized all of its memory at start-up and treats a later
 * cudaMalloc as a bug, a component embedded in a host application that owns the
 * allocator, a real-time loop that cannot take the implicit device synchronisation an
 * allocation may cause.  Such callers can still pass inputs and outputs they already
 * hold, but have nowhere to get a workspace from.
 *
 * The scratch (work counter, window cos/sin tables, rotated queries or per-split partial results) is a
 * fixed array of PC_STATIC_SCRATCH_BYTES inside the library image.  Consequences:
 *   - every GPU on which the library is loaded gives up that much memory until the
 *     process exits, whether or not this call is ever used;
 *   - a shape whose pc_parallel_attn_workspace_bytes exceeds the array is refused with
 *     PC_ERR_SCRATCH_LIMIT before anything is launched (B = 1 with tens of thousands of
 *     cached keys splits widely and can exceed it; so can a large batch, whose rotated
 *     window queries live there: B * w * Hq * d * 2 bytes);
 *   - all calls on a device share the one array and it keeps whatever the previous
 *     call left there.  The call clears the part that has to start at zero (the work
 *     counter) on `stream` itself.  Two calls whose kernels can overlap on the GPU
 *     (different streams, or different host threads on different streams) race on the
 *     array: serialise them on one stream or with events;
 *   - the first call on each device looks up the array's device address (a host-side
 *     query, no allocation call, no launch; where the CUDA runtime loads modules lazily this
 *     is also when the driver binds the array's memory on that device).  Make that first call outside of any stream
 *     capture; later calls on that device skip the query.
 *     The address is remembered per device ordinal for the life of the process: after a
 *     cudaDeviceReset, or under a context other than the device's primary one, it is stale
 *     and this entry point must not be used.
 * The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 * Arguments, layouts, status word and return values otherwise as for pc_parallel_attn.
 */
#define PC_STATIC_SCRATCH_BYTES (16u << 20)

PC_API size_t pc_parallel_attn_static_scratch_bytes(void);

PC_API int32_t pc_parallel_attn_static(int32_t B, int32_t w, int32_t Hq, int32_t Hkv, int32_t d, int32_t Nk,
                                const void* q_win, int32_t q_pos0, float rope_theta, float softmax_scale,
                                const void* k_cache, const void* v_cache, const void* k_win, const void* v_win,
                                void* out, float* lse_out, int32_t* status_word, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PC_H_ */

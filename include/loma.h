/*
 * loma.h -- C ABI of the LoMA (Lossless Compressed Memory Attention,
 * arxiv 2401.09486) attention hot path for NVIDIA B200 (sm_100a).
 *
 * The device operations and the two integer index maps:
 *
 *   loma_masked_attn_fwd   zone-masked attention over the training layout
 *                          (Section 4.3, Eq. 1-3; Section 4.4, Eq. 5-7)
 *   loma_masked_attn_bwd   its gradients with respect to q, k and v
 *                          (Section 4.4, the paths to Eq. 10)
 *   loma_rope_apply        rotary embedding of q and k at the position ids of
 *                          Section 4.5 (Eq. 14)
 *   loma_prefill_cache     the cache a one-pass prompt prefill leaves behind
 *   loma_decode_attn_ragged, loma_compress_step_ragged
 *                          the two generation steps for batches whose sequences
 *                          stand at different points of their chunks
 *   loma_decode_attn_paged, loma_compress_step_paged
 *                          the same over a pool of cache pages and a block table
 *   loma_decode_attn       one generated token over the compressed cache
 *                          (Section 3.1 steps 1 and 3; Appendix A, inference_input)
 *   loma_compress_step     the t <m> queries over the uncompressed tail, fused
 *                          with the in-place compaction of the cache
 *                          (Section 3.1 steps 2-3; Appendix A, compress_last_chunk)
 *   loma_layout_index      row -> (chunk, zone, offset, source token, position id)
 *                          (Section 4.1; Section 4.5, Eq. 14)
 *   loma_generation_index  generated token -> cache slot / position / compress flag
 *                          (Section 3.1; Appendix A, add_token_ids)
 *
 * Notation (Section 3.1, Section 4.3):  c = compression ratio, t = memory-zone
 * length, tc = t*c = reading-zone length = repetition-zone length,
 * s = t*(2c+1) = chunk length.  A laid-out sequence is n_chunks chunks
 * [tc reading | t memory | tc repetition] followed by tail_read extra reading
 * rows (an unfinished chunk); S = n_chunks*s + tail_read.
 *
 * Conventions common to every entry point
 *   - Return value: LOMA_OK (0) or a negative loma_status.  Nothing throws,
 *     aborts or traps the device.  Arguments are validated on the host before
 *     anything is launched; on error nothing has been launched.
 *   - Pointers marked [device] are CUDA device pointers on the current device;
 *     [host] are ordinary host pointers.  The caller owns every buffer before
 *     and after the call; the library allocates no device memory and reads or
 *     writes nothing through a pointer after the work enqueued by the call has
 *     finished (the tensor-core paths remember the last call's addresses, as
 *     numbers, to reuse its TMA descriptors when the same tensors come again).
 *   - stride_b / stride_h of 0 are rejected (INVALID_ARG) when B / H exceeds 1.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *     work is enqueued on it and the call returns without synchronising.
 *   - Tensors are row-major with the head dimension D contiguous.  D is 64 or
 *     128.  dtype is LOMA_F32 or LOMA_BF16 for every tensor of the call;
 *     accumulation and softmax are always fp32; bf16 outputs are rounded to
 *     nearest even.  Log-sum-exp outputs are fp32, natural log, and may be NULL.
 *   - softmax_scale <= 0 selects 1/sqrt(D) (the factor Section 4.4 drops
 *     "without loss of generality").
 *   - A mask value of 0 removes the key from the softmax (its weight is exactly
 *     zero), as the Fig. 5 caption describes.
 *   - Results are bitwise repeatable for fixed arguments.
 *   - Kernels that wait (on an mbarrier) do so with an iteration limit; on
 *     expiry they record LOMA_ERR_TIMEOUT in a device status word and return.
 *     loma_device_status() reads that word.
 */
#ifndef LOMA_H_
#define LOMA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LOMA_API __attribute__((visibility("default")))
#else
#define LOMA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LOMA_OK = 0,
    LOMA_ERR_INVALID_ARG = -1, /* NULL pointer, negative size, tc != c*t, ...        */
    LOMA_ERR_UNSUPPORTED = -2, /* D not in {64,128}, unknown dtype, device not sm_100 */
    LOMA_ERR_ALIGNMENT = -3,   /* pointer or stride not 16-byte aligned              */
    LOMA_ERR_CAPACITY = -4,    /* cache capacity too small for the request           */
    LOMA_ERR_WORKSPACE = -5,   /* workspace NULL or smaller than *_workspace_bytes    */
    LOMA_ERR_CUDA = -6,        /* a CUDA runtime/driver call failed                  */
    LOMA_ERR_TIMEOUT = -7      /* a bounded device-side wait expired                 */
} loma_status;

typedef enum { LOMA_F32 = 0, LOMA_BF16 = 1 } loma_dtype;

enum {
    /* Section 4.3 criterion 2 and Eq. 3 (memory rows all zero) say that memory
     * rows see only their own reading zone and their own memory zone, and
     * Appendix A hands the compress pass only the last tc cache entries.  That
     * is the default.  With this flag memory rows additionally see every earlier
     * memory zone (masked forward) and the compress pass additionally attends to
     * the mem_len memory entries already in the cache; both change together so
     * that incremental generation still equals the one-shot forward. */
    LOMA_FLAG_MEM_SEES_PRIOR_MEM = 1u,
    /* Inference layout: chunks are [tc reading | t memory] with no repetition zone (s = tc + t), the
     * sequence Section 3.1 / Appendix A actually feed the model -- the <r> rows exist only for the
     * training loss (Section 4.2).  The mask is Eq. 2 with the repetition rows and columns deleted.
     * One pass of loma_masked_attn_fwd over a prompt laid out this way equals ingesting the prompt
     * token by token with a compress pass per chunk. */
    LOMA_FLAG_NO_REP_ZONE = 2u,
    /* Run the plain CUDA-core kernel even where a tensor-core kernel exists
     * (second opinion for tests; always used for LOMA_F32). */
    LOMA_FLAG_FORCE_GENERIC = 1u << 8
};

/* Zone codes written by loma_layout_index. */
enum { LOMA_ZONE_READ = 0, LOMA_ZONE_MEM = 1, LOMA_ZONE_REP = 2 };

/* ---------------------------------------------------------------------------
 * loma_layout_index -- Section 4.1 (chunk layout) and Eq. 14 (position ids).
 *
 * For every row i of a laid-out sequence of S = n_chunks*t*(2c+1) + tail_read
 * rows writes
 *   chunk[i]      y = i div s                       (tail rows: n_chunks)
 *   zone[i]       LOMA_ZONE_READ / _MEM / _REP
 *   offset[i]     position inside the zone
 *   src_token[i]  y*tc + offset for reading rows (the original token carried)
 *                 and repetition rows (the token to reproduce, Eq. 13);
 *                 -1 for <m> rows
 *   pos_id[i]     reading rows: y*tc + offset (original ids are preserved);
 *                 memory row j: y*tc + (j+1)*c - 1 (Eq. 14, chunk start y*tc as
 *                 in the Appendix A listing); repetition rows: y*tc + offset
 *                 (the paper does not say; same id as the token reproduced).
 * Each output is int32[S]; any of them may be NULL (skipped).  on_device != 0:
 * outputs are [device] and filled by a kernel on `stream`; on_device == 0:
 * outputs are [host], filled synchronously, no CUDA call is made.
 * flags: LOMA_FLAG_NO_REP_ZONE selects the layout without repetition zones (S = n_chunks*t*(c+1) + tail_read).
 * t == 0 requires n_chunks == 0 (the sequence is one reading zone).
 * Errors: INVALID_ARG (negative sizes, c < 1, t == 0 with n_chunks > 0,
 * t > 0 with tail_read > tc, S > INT32_MAX), CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_layout_index(int n_chunks, int c, int t, int tail_read, unsigned flags,
                               int32_t* chunk, int32_t* zone, int32_t* offset,
                               int32_t* src_token, int32_t* pos_id,
                               int on_device, void* stream);

/* ---------------------------------------------------------------------------
 * loma_generation_index -- Section 3.1 steps 1-3, Appendix A add_token_ids.
 *
 * For generated token g = 0..n_tokens-1 (no prompt), with the cache holding
 * compressed_chunks*t memory entries followed by the uncompressed tail:
 *   slot[g]            cache index the token's K/V is appended at
 *                      = (g div tc)*t + g mod tc   (= g when t == 0)
 *   pos_id[g]          g (the generator's cursor)
 *   compress_after[g]  1 if the tail reaches tc with this token, i.e. a compress
 *                      pass follows it; always 0 when t == 0
 * Outputs int32[n_tokens], NULL = skipped; on_device as above.
 * Errors: INVALID_ARG, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_generation_index(int n_tokens, int c, int t,
                                   int32_t* slot, int32_t* pos_id, int32_t* compress_after,
                                   int on_device, void* stream);

/* ---------------------------------------------------------------------------
 * loma_masked_attn_fwd -- O = Softmax(A) V with A = scale * Q K^T restricted to
 * the mask M of Eq. 2 (diagonal blocks Eq. 1, sub-diagonal blocks Eq. 3),
 * evaluated row by row as in Eq. 7.  The mask is never stored: it is computed
 * from (chunk, zone, offset) of the row and the key, and tiles with no allowed
 * entry are skipped.
 *
 *   q, k, v [device, in]   [B, H, S, D], element (b,h,i,d) at
 *                          b*stride_b + h*stride_h + i*stride_s + d  (elements)
 *   o       [device, out]  same shape and strides as q
 *   lse     [device, out]  fp32 [B, H, S] contiguous, or NULL
 *   n_chunks, c, t, tc, tail_read   layout; tc must equal c*t; t == 0 requires
 *                          n_chunks == 0 and gives plain causal attention over
 *                          tail_read rows; t > 0 requires tail_read <= tc
 *   flags                  LOMA_FLAG_* bits
 * o must not alias q, k or v.  Rows are independent; every row has at least one
 * allowed key (itself), so no output is undefined.
 * Concurrency: the bf16 kernel hands out its tiles from a counter inside the library.
 * Calls on different streams each use their stream's own counter and may overlap freely
 * (the first 192 streams that call get one; later ones run with a fixed deal of the
 * tiles, slower by a few percent on short layouts).  A call recorded while its stream is
 * being captured into a CUDA graph gets a counter of its own for good (320 per device,
 * then the fixed deal), so replays may overlap eager calls and other graphs; two
 * replays of the same captured call must not overlap each other (CUDA already orders
 * launches of one executable graph).  Make one eager bf16 call per device before the
 * first capture: the first call looks up device symbols and sets kernel attributes.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT (pointers and byte strides must be
 * multiples of 16), CUDA.  S == 0 or B*H == 0 is a successful no-op.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_masked_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                                  int B, int H, int D,
                                  int n_chunks, int c, int t, int tc, int tail_read,
                                  int64_t stride_b, int64_t stride_h, int64_t stride_s,
                                  loma_dtype dtype, float softmax_scale, unsigned flags, void* stream);

/* ---------------------------------------------------------------------------
 * loma_masked_attn_bwd -- gradients of loma_masked_attn_fwd: the chain rule through
 * O = Softmax(A) V of Eq. 7, the paths Section 4.4 follows to Eq. 10 (a loss on the
 * repetition rows reaches k_m and v_m).  With P_ij = exp(scale q_i.k_j - lse_i) on the
 * entries Eq. 2 allows and dA_ij = P_ij (dO_i.v_j - dO_i.O_i):
 *      dQ = scale dA K      dK = scale dA^T Q      dV = P^T dO
 * Blocked entries carry no gradient.  Every output row is produced by one owner in a fixed
 * order (no atomics): results repeat bit for bit.
 *
 *   q, k, v, o, d_o [device, in]   [B, H, S, D] with the strides of loma_masked_attn_fwd;
 *                                  o and lse are the forward's outputs for these q, k, v
 *   lse             [device, in]   fp32 [B, H, S] contiguous (natural-log normaliser)
 *   dq, dk, dv      [device, out]  same shape, strides and dtype as q; must not alias an input
 *   workspace       [device]       at least loma_masked_attn_bwd_workspace_bytes(...) bytes,
 *                                  256-byte aligned; contents need not be initialised
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE, CUDA.  S == 0 or B*H == 0 is a no-op.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_masked_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                  const float* lse, void* dq, void* dk, void* dv,
                                  int B, int H, int D,
                                  int n_chunks, int c, int t, int tc, int tail_read,
                                  int64_t stride_b, int64_t stride_h, int64_t stride_s,
                                  loma_dtype dtype, float softmax_scale, unsigned flags,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* Workspace size in bytes for loma_masked_attn_bwd (0 for an invalid layout). */
LOMA_API size_t loma_masked_attn_bwd_workspace_bytes(int B, int H, int D, int n_chunks, int c, int t, int tail_read,
                                                     unsigned flags);

/* ---------------------------------------------------------------------------
 * loma_rope_apply -- rotary position embedding of Q and K, in place, at the position ids of
 * Section 4.5: reading rows keep their original ids, memory row j of chunk y gets
 * y*tc + (j+1)c - 1 (Eq. 14; the generator's position_type 'intermittent'), repetition rows the id
 * of the token they reproduce (the paper does not say).  position_type 1 selects the generator's
 * other setting (Appendix A): memory row j of chunk y gets y*t + j.  The ids are computed from the
 * row number; no id tensor is read.  The paper passes its ids to a Llama-2 model and does not write
 * the rotation out; this is that model's: with half = D/2, theta_d = theta_base^(-2d/D),
 *     x'[d] = x[d] cos(p theta_d) - x[d+half] sin(p theta_d),
 *     x'[d+half] = x[d+half] cos(p theta_d) + x[d] sin(p theta_d),      d in [0, half).
 *
 * Adding LOMA_ROPE_INVERSE (2) to position_type rotates by the opposite angle: the inverse, which is also the
 * transpose, i.e. what the gradients of the rotated q and k need on their way back to the unrotated ones.
 *
 *   q, k [device, in/out]  [B, H, S, D] with the strides of loma_masked_attn_fwd; either may be NULL
 *   theta_base             <= 0 selects 10000
 *   flags                  LOMA_FLAG_NO_REP_ZONE for the layout without repetition zones
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.  S == 0 or B*H == 0 is a no-op.
 * ------------------------------------------------------------------------- */
enum { LOMA_ROPE_INVERSE = 2 };

LOMA_API int loma_rope_apply(void* q, void* k, int B, int H, int D,
                             int n_chunks, int c, int t, int tc, int tail_read,
                             int64_t stride_b, int64_t stride_h, int64_t stride_s,
                             loma_dtype dtype, float theta_base, int position_type, unsigned flags, void* stream);

/* ---------------------------------------------------------------------------
 * loma_prefill_cache -- what the cache holds after a prompt has been ingested (Section 3.1 step 3
 * applied to every complete chunk; Appendix A, compress_last_chunk's torch.cat lines): the memory-zone
 * K/V rows of chunks 0..n_chunks-1 in order, followed by the tail_read rows of the unfinished chunk.
 * Bit-exact gather from the laid-out K and V of a one-pass prefill into the generation cache.
 *
 *   k, v             [device, in]   [B, H, S, D] with the strides of loma_masked_attn_fwd
 *   k_cache, v_cache [device, out]  [B, H, cap, D] contiguous; entries [0, n_chunks*t + tail_read) are
 *                                   written, nothing else is touched
 *   flags            LOMA_FLAG_NO_REP_ZONE if k, v are in the layout without repetition zones
 * Returns the new valid cache length in *cache_len_out ([host], may be NULL).
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY (cap < n_chunks*t + tail_read), CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_prefill_cache(const void* k, const void* v, void* k_cache, void* v_cache,
                                int B, int H, int D, int cap,
                                int n_chunks, int c, int t, int tc, int tail_read,
                                int64_t stride_b, int64_t stride_h, int64_t stride_s,
                                loma_dtype dtype, unsigned flags, int* cache_len_out, void* stream);

/* ---------------------------------------------------------------------------
 * loma_masked_attn_plan_coverage -- host-only introspection of the tensor-core
 * kernel's tile plan for loma_masked_attn_fwd (Eq. 1-3).  The kernel never
 * stores the mask: it visits, per 128-row query tile, only the key tiles that
 * hold an allowed entry, and inside a visited tile lets each row attend to one
 * interval of columns.  This routine replays that plan on the host and writes
 *   counts[i*S + j] = how many visits let row i attend to column j  (saturating)
 * into a [host] uint8 buffer of S*S bytes, S = n_chunks*t*(2c+1) + tail_read.
 * A correct plan reproduces the mask M of Eq. 2 exactly (every count 0 or 1).
 * No CUDA call is made.  Errors: INVALID_ARG (bad geometry, NULL, S*S > 2^32).
 * ------------------------------------------------------------------------- */
LOMA_API int loma_masked_attn_plan_coverage(int n_chunks, int c, int t, int tail_read, unsigned flags,
                                            uint8_t* counts);

/* ---------------------------------------------------------------------------
 * loma_masked_attn_bwd_plan_coverage -- the same host-only replay for the pass of
 * loma_masked_attn_bwd that produces dK and dV.  That pass owns one 128-row key tile at a
 * time and walks the query tiles that may attend to it (the columns of Eq. 2 read
 * downwards); inside a visited query tile each key lets one interval of rows through.
 * counts has the layout of loma_masked_attn_plan_coverage and must again equal M of Eq. 2.
 * No CUDA call is made.  Errors: INVALID_ARG.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_masked_attn_bwd_plan_coverage(int n_chunks, int c, int t, int tail_read, unsigned flags,
                                                uint8_t* counts);

/* ---------------------------------------------------------------------------
 * loma_decode_attn -- one new token per (batch, head) attends to the cache_len
 * entries already in the cache (all memory entries, then the uncompressed tail)
 * and to itself: the mask row tril(ones(1, 1+k), diagonal=k) of Appendix A with
 * k = cache_len.  Its key and value are appended at slot cache_len.
 *
 *   q               [device, in]      [B, H, 1, D] contiguous
 *   k_new, v_new    [device, in]      [B, H, 1, D] contiguous; both NULL means the
 *                                     token's K/V already sit at slot cache_len
 *   k_cache, v_cache [device, in/out] [B, H, cap, D] contiguous; entries
 *                                     [0, cache_len) are read, entry cache_len is
 *                                     written (when k_new is given); nothing else
 *                                     is touched
 *   o               [device, out]     [B, H, 1, D] contiguous
 *   lse             [device, out]     fp32 [B, H], or NULL
 *   cache_len       entries before this token, the same for every (b,h);
 *                   requires 0 <= cache_len < cap
 *   workspace       [device] scratch of at least
 *                   loma_decode_workspace_bytes(B,H,D,cache_len) bytes, 16-byte
 *                   aligned; contents on entry and exit are unspecified
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY (cache_len >= cap),
 * WORKSPACE, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn(const void* q, const void* k_new, const void* v_new,
                              void* k_cache, void* v_cache, void* o, float* lse,
                              int B, int H, int D, int cap, int cache_len,
                              loma_dtype dtype, float softmax_scale, unsigned flags,
                              void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * The rope-fused steps for ragged batches and the paged cache: loma_decode_attn_rope /
 * loma_compress_step_rope (Section 4.5; Appendix A position ids) with one position per
 * sequence, since every sequence of a ragged batch has its own `cursor`.
 *
 *   positions [device, in]  int32 [B]: the position id of sequence b's new token
 *   pos0s     [device, in]  int32 [B]: the id of sequence b's memory row 0; row j gets
 *                           pos0s[b] + j * pos_stride (entries of sequences that do not compress
 *                           in this call, mem_lens[b] < 0, are ignored)
 * Every other argument, and every rule, is that of the entry point without `_rope`; k_new and
 * v_new are required.  Errors: those of that entry point, plus INVALID_ARG (NULL positions,
 * negative stride), ALIGNMENT (positions not 4-byte aligned), UNSUPPORTED (memory zone too long
 * to stage, t*D*sizeof(element) > 200 KB).
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn_ragged_rope(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                          void* v_cache, void* o, float* lse, int B, int H, int D, int cap,
                                          const int32_t* cache_lens, int max_cache_len, const int32_t* positions,
                                          float theta_base, loma_dtype dtype, float softmax_scale, unsigned flags,
                                          void* workspace, size_t workspace_bytes, void* stream);
LOMA_API int loma_decode_attn_paged_rope(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                                         const int32_t* block_table, void* o, float* lse, int B, int H, int D,
                                         int page_size, int max_pages, int n_pages, const int32_t* cache_lens,
                                         int max_cache_len, const int32_t* positions, float theta_base, loma_dtype dtype,
                                         float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes,
                                         void* stream);
LOMA_API int loma_compress_step_ragged_rope(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache,
                                            void* v_cache, void* o_mem, float* lse, int B, int H, int D, int cap,
                                            const int32_t* mem_lens, int max_mem_len, int c, int t, int tc,
                                            const int32_t* pos0s, int pos_stride, float theta_base, loma_dtype dtype,
                                            float softmax_scale, unsigned flags, void* stream);
LOMA_API int loma_compress_step_paged_rope(const void* q_mem, const void* k_mem, const void* v_mem, void* k_pool,
                                           void* v_pool, const int32_t* block_table, void* o_mem, float* lse, int B, int H,
                                           int D, int page_size, int max_pages, int n_pages, const int32_t* mem_lens,
                                           int max_mem_len, int c, int t, int tc, const int32_t* pos0s, int pos_stride,
                                           float theta_base, loma_dtype dtype, float softmax_scale, unsigned flags,
                                           void* stream);

/* ---------------------------------------------------------------------------
 * loma_decode_attn_layers, loma_compress_step_layers -- the generator's loop over the layers of the
 * model (Appendix A: inference_input hands every layer's cache to the model, compress_last_chunk
 * slices and re-concatenates `for i in range(len(self.kv_cache))`): the same step for n_layers
 * independent (q, k, v, cache, output) sets of one shape, enqueued back to back on the stream.
 * Every pointer argument is a [host] array of n_layers [device] pointers with the meaning the
 * single-layer call gives them (k_new / v_new / lse may be NULL as a whole, or hold NULL entries
 * where the single-layer call allows NULL).  The layers share one workspace of the single-layer
 * size: they run one after the other.  Caches and outputs of different layers must be distinct.
 * All layers are validated before the first is enqueued.  Errors: those of the single-layer call.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn_layers(int n_layers, const void* const* q, const void* const* k_new,
                                     const void* const* v_new, void* const* k_cache, void* const* v_cache,
                                     void* const* o, float* const* lse, int B, int H, int D, int cap, int cache_len,
                                     loma_dtype dtype, float softmax_scale, unsigned flags, void* workspace,
                                     size_t workspace_bytes, void* stream);
LOMA_API int loma_compress_step_layers(int n_layers, const void* const* q_mem, const void* const* k_mem,
                                       const void* const* v_mem, void* const* k_cache, void* const* v_cache,
                                       void* const* o_mem, float* const* lse, int B, int H, int D, int cap, int mem_len,
                                       int c, int t, int tc, loma_dtype dtype, float softmax_scale, unsigned flags,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * loma_decode_attn_rope, loma_compress_step_rope -- the two generation steps with the rotary
 * position embedding of Section 4.5 done inside the step: q and the new key(s) are rotated in
 * registers / shared memory by their position ids right where the kernels load them, so the
 * generation loop has no separate rotation pass (the training layout is rotated by
 * loma_rope_apply).  The rotation is the one loma_rope_apply documents (feature d paired with
 * d + D/2, angle pos * theta_base^(-2d/D), theta_base <= 0 selects 10000).  The rotated keys,
 * rounded to the storage type, are what the step attends to and what is written to the cache;
 * values are not rotated.  Everything else is as in loma_decode_attn / loma_compress_step.
 *
 *   decode:    pos = the token's position id -- the generator's `cursor` (Appendix A,
 *              inference_input: position_ids = arange(cursor, cursor + l)); k_new and v_new
 *              are required
 *   compress:  memory row j gets pos0 + j * pos_stride: Eq. 14 ('intermittent') is
 *              pos0 = y*tc + c - 1, pos_stride = c for chunk y; the generator's other setting
 *              is pos0 = mem_len (= mem_cursor), pos_stride = 1 (Appendix A, compress_last_chunk)
 * Errors: as the plain calls, plus INVALID_ARG for a negative position or missing k_new, and
 * UNSUPPORTED for a memory zone too long to stage (t*D*sizeof(element) > 200 KB).
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn_rope(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                   void* o, float* lse, int B, int H, int D, int cap, int cache_len, int pos,
                                   float theta_base, loma_dtype dtype, float softmax_scale, unsigned flags,
                                   void* workspace, size_t workspace_bytes, void* stream);
LOMA_API int loma_compress_step_rope(const void* q_mem, const void* k_mem, const void* v_mem, void* k_cache,
                                     void* v_cache, void* o_mem, float* lse, int B, int H, int D, int cap, int mem_len,
                                     int c, int t, int tc, int pos0, int pos_stride, float theta_base, loma_dtype dtype,
                                     float softmax_scale, unsigned flags, void* workspace, size_t workspace_bytes,
                                     void* stream);

/* ---------------------------------------------------------------------------
 * loma_prefill_attn -- several new tokens at once over an existing cache: Appendix A,
 * `inference_input` called with l > 1 tokens, which `add_token_ids` does whenever a
 * prompt (or a piece of one) arrives while the cache already holds entries: it feeds
 * exactly as many tokens as fill the uncompressed tail up to tc, then compresses.  The
 * mask is the listing's tril(ones(l, l + cache_len), diagonal = cache_len): new token i
 * sees every cached entry and new tokens 0 .. i.  The l new K/V rows are appended to the
 * cache first (bit-exact), at entries [cache_len, cache_len + l).  With l == 1 this is
 * loma_decode_attn; with cache_len == 0 plain causal attention.
 *
 *   q, k_new, v_new [device, in]      [B, H, l, D] contiguous; k_new and v_new may both be
 *                                     NULL when the new rows are already in the cache
 *   k_cache, v_cache [device, in/out] [B, H, cap, D] contiguous; entries [0, cache_len) are
 *                                     read, [cache_len, cache_len + l) written then read
 *   o                [device, out]    [B, H, l, D] contiguous
 *   lse              [device, out]    fp32 [B, H, l] or NULL
 *   cache_len        entries before this call (memory entries + uncompressed tail), the
 *                    same for every sequence of the batch
 * bf16 calls with l >= 8 run on the tensor-core kernel of loma_masked_attn_fwd (its
 * concurrency notes apply), the rest on CUDA cores.  No workspace.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY (cache_len + l > cap), CUDA.
 * l == 0 or B*H == 0 is a successful no-op.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_prefill_attn(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                               void* o, float* lse, int B, int H, int D, int l, int cap, int cache_len,
                               loma_dtype dtype, float softmax_scale, unsigned flags, void* stream);

/* ---------------------------------------------------------------------------
 * loma_prefill_attn_ragged, loma_prefill_attn_paged -- the same step (Appendix A,
 * `inference_input` with l > 1 tokens) for a batch whose sequences hold different numbers
 * of entries, over a contiguous or a paged cache: one run of the generator per sequence,
 * each feeding l tokens.  Sequence b appends its l rows at entries
 * [cache_lens[b], cache_lens[b] + l) and its new token i sees entries 0 .. cache_lens[b] + i.
 *
 *   cache_lens [device, in]  int32 [B]: entries of every sequence before the call; values are
 *                            clamped to [0, max_cache_len] on the device
 *   max_cache_len            a bound on cache_lens that the caller vouches for (work is sized by it)
 *   ragged: k_cache, v_cache [B, H, cap, D] as in loma_prefill_attn.  bf16 calls with l >= 8 run on
 *           the tensor-core kernel; for them the call also sets the entries from each
 *           sequence's new end up to the next multiple of 128 (at most cap) to zero: that
 *           kernel reads them (with weight zero), and the contents of the cache past a
 *           sequence's valid length are unspecified anyway.
 *   paged:  k_pool, v_pool [n_pages, H, page_size, D] and block_table int32 [B, max_pages] as in
 *           loma_decode_attn_paged (page numbers clamped to the pool).  bf16 calls with l >= 8 over
 *           pages of a multiple of 128 rows run on the tensor-core kernel (a 128-key tile then lies
 *           in one page; the zeroing described above applies, inside the sequence's last page);
 *           every other call on CUDA cores, one warp per new row.
 * Other arguments, outputs and errors as loma_prefill_attn; CAPACITY when max_cache_len + l
 * exceeds cap (ragged) or max_pages * page_size (paged); INVALID_ARG for a missing table or
 * length array or a page size that is not a power of two.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_prefill_attn_ragged(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                      void* v_cache, void* o, float* lse, int B, int H, int D, int l, int cap,
                                      const int32_t* cache_lens, int max_cache_len, loma_dtype dtype,
                                      float softmax_scale, unsigned flags, void* stream);
LOMA_API int loma_prefill_attn_paged(const void* q, const void* k_new, const void* v_new, void* k_pool, void* v_pool,
                                     const int32_t* block_table, void* o, float* lse, int B, int H, int D, int l,
                                     int page_size, int max_pages, int n_pages, const int32_t* cache_lens,
                                     int max_cache_len, loma_dtype dtype, float softmax_scale, unsigned flags,
                                     void* stream);

/* ---------------------------------------------------------------------------
 * loma_prefill_attn_rope, loma_prefill_attn_ragged_rope, loma_prefill_attn_paged_rope -- the
 * prompt piece with the rotary embedding of Section 4.5 fused in (rotation as in
 * loma_rope_apply): new token i of a sequence is rotated by the id pos0 + i -- Appendix A,
 * `inference_input`: position_ids = cursor .. cursor + l - 1, the count of tokens seen so
 * far, not the cache length.  q is rotated on its way into the step (the caller's q is
 * left as it is; o serves as the scratch for the rotated queries before it receives the
 * output); k_new is rotated, rounded to the storage type and appended -- the cache holds
 * rotated keys, as after loma_decode_attn_rope; v_new is appended as it is.
 *
 *   pos0                   id of the piece's first token, the same for every sequence
 *   positions [device, in] ragged / paged: int32 [B], the id of every sequence's first new token
 *   theta_base             <= 0 selects 10000
 * k_new and v_new are required.  Everything else, and the errors, as the entry point
 * without the suffix; INVALID_ARG also for a negative pos0, an id that would pass
 * INT_MAX, or a missing positions array.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_prefill_attn_rope(const void* q, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                    void* o, float* lse, int B, int H, int D, int l, int cap, int cache_len, int pos0,
                                    float theta_base, loma_dtype dtype, float softmax_scale, unsigned flags,
                                    void* stream);
LOMA_API int loma_prefill_attn_ragged_rope(const void* q, const void* k_new, const void* v_new, void* k_cache,
                                           void* v_cache, void* o, float* lse, int B, int H, int D, int l, int cap,
                                           const int32_t* cache_lens, int max_cache_len, const int32_t* positions,
                                           float theta_base, loma_dtype dtype, float softmax_scale, unsigned flags,
                                           void* stream);
LOMA_API int loma_prefill_attn_paged_rope(const void* q, const void* k_new, const void* v_new, void* k_pool,
                                          void* v_pool, const int32_t* block_table, void* o, float* lse, int B, int H,
                                          int D, int l, int page_size, int max_pages, int n_pages,
                                          const int32_t* cache_lens, int max_cache_len, const int32_t* positions,
                                          float theta_base, loma_dtype dtype, float softmax_scale, unsigned flags,
                                          void* stream);

/* Host-only replay of the tile plan the tensor-core kernel follows for loma_prefill_attn
 * (Appendix A, inference_input mask): counts[i*(cache_len+l) + j] = number of visits in
 * which new token i attends to key j, into a [host] uint8 buffer of l*(cache_len+l) bytes.
 * A correct plan gives tril(ones(l, l+cache_len), diagonal=cache_len) exactly.  No CUDA call.
 * Errors: INVALID_ARG. */
LOMA_API int loma_prefill_attn_plan_coverage(int l, int cache_len, uint8_t* counts);

LOMA_API size_t loma_decode_workspace_bytes(int B, int H, int D, int cache_len);

/* ---------------------------------------------------------------------------
 * loma_decode_attn_ragged -- the same decode step for a batch whose sequences stand at
 * different points of their chunks.  The generator of Appendix A handles one sequence;
 * batched, each sequence b has its own count of cache entries (memory entries of its
 * compressed chunks plus its current tail), so sequence b attends to cache[b][0, len_b) and
 * to itself, and its K/V are appended at slot len_b.
 *
 *   cache_lens     [device, in]  int32 [B]: entries before this token, per sequence;
 *                                values are clamped to [0, max_cache_len] on the device
 *   max_cache_len  [host]        an upper bound of cache_lens known to the caller without a
 *                                device read (e.g. the longest sequence's length); sizes the
 *                                launch and the workspace: loma_decode_workspace_bytes(B,H,D,max_cache_len);
 *                                requires 0 <= max_cache_len < cap
 * Everything else as in loma_decode_attn.  The split of the key range depends on
 * max_cache_len only, so results repeat bit for bit for fixed arguments.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY, WORKSPACE, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn_ragged(const void* q, const void* k_new, const void* v_new,
                                     void* k_cache, void* v_cache, void* o, float* lse,
                                     int B, int H, int D, int cap,
                                     const int32_t* cache_lens, int max_cache_len,
                                     loma_dtype dtype, float softmax_scale, unsigned flags,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * loma_decode_attn_paged -- the ragged decode step over a paged cache: the K and V entries of all
 * sequences live in one pool of fixed-size pages, and a block table says which page holds which
 * stretch of which sequence (the paper keeps one contiguous cache per sequence; this is the same
 * step, Appendix A inference_input, for a serving engine that hands out cache memory page by page).
 * Slot j of sequence b is row j % page_size of page block_table[b][j / page_size].
 *
 *   k_pool, v_pool [device, in/out]  [n_pages, H, page_size, D] contiguous
 *   block_table    [device, in]      int32 [B, max_pages]; entries are clamped to [0, n_pages) on the device;
 *                                    only the blocks below a sequence's length (and the one that takes the new
 *                                    token) are read
 *   page_size      a power of two
 *   cache_lens, max_cache_len        as in loma_decode_attn_ragged; max_cache_len < max_pages * page_size
 * The new token's K/V are written at slot cache_lens[b] of sequence b (its page must be in the table).
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY, WORKSPACE, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn_paged(const void* q, const void* k_new, const void* v_new,
                                    void* k_pool, void* v_pool, const int32_t* block_table,
                                    void* o, float* lse, int B, int H, int D,
                                    int page_size, int max_pages, int n_pages,
                                    const int32_t* cache_lens, int max_cache_len,
                                    loma_dtype dtype, float softmax_scale, unsigned flags,
                                    void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * loma_compress_step_paged -- loma_compress_step_ragged over the paged cache of
 * loma_decode_attn_paged: sequence b (when mem_lens[b] >= 0) reads its tail from slots
 * [mem_lens[b], mem_lens[b] + tc) through the block table and its t memory keys and values are
 * written over slots [mem_lens[b], mem_lens[b] + t), wherever their pages lie.  Afterwards the
 * sequence's valid length is mem_lens[b] + t; pages that hold only slots beyond it can go back to
 * the caller's allocator (the library never touches the table).
 * Default mask only (LOMA_FLAG_MEM_SEES_PRIOR_MEM returns UNSUPPORTED).  No workspace.
 * Requires max_mem_len + tc <= max_pages * page_size.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_compress_step_paged(const void* q_mem, const void* k_mem, const void* v_mem,
                                      void* k_pool, void* v_pool, const int32_t* block_table,
                                      void* o_mem, float* lse, int B, int H, int D,
                                      int page_size, int max_pages, int n_pages,
                                      const int32_t* mem_lens, int max_mem_len, int c, int t, int tc,
                                      loma_dtype dtype, float softmax_scale, unsigned flags, void* stream);

/* ---------------------------------------------------------------------------
 * loma_decode_attn_static -- the same decode step as loma_decode_attn (bf16
 * only), for callers that cannot hand the library a workspace because they
 * cannot obtain device memory at the point of the call.  (The paper has no
 * counterpart: this is a packaging variant, not a different computation.)
 *
 * Who needs it: code that runs after the process has committed all of its
 * device memory to a fixed plan (a serving engine whose KV-cache pool owns the
 * rest of HBM, so a late cudaMalloc fails); plug-ins called from a host
 * runtime that forbids allocation inside its step function because
 * cudaMalloc/cudaFree synchronise the whole device; and callers with no
 * allocator of their own at hand (a bare C program holding only the tensors
 * it was given).  For them the split-KV partial results go into an 8 MiB
 * array that is part of the library image itself:
 *
 *   - Every GPU on which the library is used holds those 8 MiB
 *     (loma_decode_static_scratch_bytes()) from the first use until the
 *     process exits, whether or not this entry point is ever called again.
 *   - A request whose partials do not fit -- i.e. whose
 *     loma_decode_workspace_bytes(B,H,D,cache_len) exceeds that size -- is
 *     rejected with LOMA_ERR_WORKSPACE and nothing is launched.  (B*H = 1024
 *     pairs at a cache length of 8k need 4.8 MB; 1024 pairs at 16k do not fit.)
 *   - The call itself allocates nothing: no cudaMalloc, cudaFree or other
 *     allocating routine is reached from it.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and caches it.  Make
 *     that first call during set-up.
 *   - All calls share the one array.  Nothing in it has to be cleared between
 *     calls (every partial that is read has been written by the same call),
 *     but two calls that can overlap on the GPU -- different streams without an
 *     ordering between them -- overwrite each other's partials and give wrong
 *     results.  Keep calls on one stream, or order them with events.
 *
 * Arguments, layouts, the append of k_new/v_new at slot cache_len and the
 * results are exactly those of loma_decode_attn without its workspace pair and
 * flags.  Errors: INVALID_ARG, UNSUPPORTED (dtype other than LOMA_BF16, D not
 * 64/128, device not sm_100), ALIGNMENT, CAPACITY, WORKSPACE (too large for the
 * built-in array), CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_decode_attn_static(const void* q, const void* k_new, const void* v_new,
                                     void* k_cache, void* v_cache, void* o, float* lse,
                                     int B, int H, int D, int cap, int cache_len,
                                     loma_dtype dtype, float softmax_scale, void* stream);

/* Size in bytes of the built-in scratch array used by loma_decode_attn_static. */
LOMA_API size_t loma_decode_static_scratch_bytes(void);

/* ---------------------------------------------------------------------------
 * loma_compress_step -- Section 3.1 step 2 (one pass of t <m> tokens over
 * KV_Read) and step 3 (KV_Read is discarded), fused.
 *
 * Precondition (asserted by the Appendix A listing): the cache holds mem_len
 * memory entries followed by exactly tc tail entries.  The t memory queries
 * attend with an all-ones t x (tc+t) mask to the tail and to their own keys
 * (with LOMA_FLAG_MEM_SEES_PRIOR_MEM also to entries [0, mem_len)).  Then the
 * cache becomes cat(cache[:mem_len], k_mem): k_mem / v_mem are copied, bit for
 * bit, into slots [mem_len, mem_len+t), overwriting the first tail entries
 * only after every read of them has completed.
 *
 *   q_mem, k_mem, v_mem [device, in]  [B, H, t, D] contiguous
 *   k_cache, v_cache [device, in/out] [B, H, cap, D] contiguous, cap >= mem_len+tc
 *   o_mem            [device, out]    [B, H, t, D] contiguous
 *   lse              [device, out]    fp32 [B, H, t], or NULL
 * Postcondition: the valid cache length is mem_len + t; entries [0, mem_len) are
 * untouched; entries at and beyond mem_len + t are unspecified.
 * Requires t >= 1, c >= 1, tc == c*t, mem_len >= 0.
 *   workspace  [device] at least loma_compress_workspace_bytes(...) bytes
 *              (NULL is accepted when that is 0)
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY, WORKSPACE, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_compress_step(const void* q_mem, const void* k_mem, const void* v_mem,
                                void* k_cache, void* v_cache, void* o_mem, float* lse,
                                int B, int H, int D, int cap, int mem_len, int c, int t, int tc,
                                loma_dtype dtype, float softmax_scale, unsigned flags,
                                void* workspace, size_t workspace_bytes, void* stream);

LOMA_API size_t loma_compress_workspace_bytes(int B, int H, int D, int t, int mem_len, unsigned flags);

/* ---------------------------------------------------------------------------
 * loma_compress_step_ragged -- the compress step for a batch whose sequences reach the end
 * of a chunk at different times (Section 3.1 steps 2-3 once per sequence; Appendix A runs one
 * sequence).  Sequence b compresses in this call iff mem_lens[b] >= 0: its t memory queries then
 * attend to its tail cache[b][mem_lens[b], mem_lens[b] + tc) and to their own keys, and
 * k_mem[b], v_mem[b] are written over slots [mem_lens[b], mem_lens[b] + t).  Sequences with a
 * negative entry are left alone: their caches and their rows of o_mem and lse are not touched.
 *
 *   mem_lens     [device, in]  int32 [B]: memory entries in front of the tail, per sequence,
 *                              or negative; values above max_mem_len are clamped to it
 *   max_mem_len  [host]        upper bound of mem_lens; requires max_mem_len + tc <= cap
 * Only the default mask (memory rows see their own chunk) is offered: with
 * LOMA_FLAG_MEM_SEES_PRIOR_MEM the call returns UNSUPPORTED.  No workspace is needed.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CAPACITY, CUDA.
 * ------------------------------------------------------------------------- */
LOMA_API int loma_compress_step_ragged(const void* q_mem, const void* k_mem, const void* v_mem,
                                       void* k_cache, void* v_cache, void* o_mem, float* lse,
                                       int B, int H, int D, int cap,
                                       const int32_t* mem_lens, int max_mem_len, int c, int t, int tc,
                                       loma_dtype dtype, float softmax_scale, unsigned flags, void* stream);

/* Synchronises `stream`, then returns the device status word of the current
 * device: LOMA_OK, or LOMA_ERR_TIMEOUT if a bounded wait inside a kernel has
 * expired since the last call (the word is cleared by the call).
 * LOMA_ERR_CUDA if the synchronisation or the read fails. */
LOMA_API int loma_device_status(void* stream);

/* Failure-detection self test: enqueues a one-thread kernel that waits, with the library's bounded
 * wait, on a barrier nobody ever signals.  After about a millisecond the wait gives up, the kernel
 * records LOMA_ERR_TIMEOUT in the device status word and returns normally (no trap, the context
 * stays usable); the next loma_device_status() then returns LOMA_ERR_TIMEOUT once.
 * Errors: UNSUPPORTED (device), CUDA. */
LOMA_API int loma_selftest_bounded_wait(void* stream);

/* Number of kernels this library has enqueued in the calling process since it
 * was loaded (all devices, all streams).  Host-side counter; never fails. */
LOMA_API uint64_t loma_launch_count(void);

/* Number of bf16 calls (forward or backward of the masked attention) for which the
 * tensor-core path declined the arguments (TMA descriptor not encodable, zone longer
 * than the tile plan supports) and the slower CUDA-core kernels ran instead.  The
 * result of such a call is still correct; a caller that cares about speed can watch
 * this counter.  Host-side counter; never fails. */
LOMA_API uint64_t loma_fallback_count(void);

/* Static, human-readable name of a status code. */
LOMA_API const char* loma_status_string(int status);

/* Library version: major*10000 + minor*100 + patch. */
LOMA_API int loma_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LOMA_H_ */

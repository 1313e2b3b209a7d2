/*
 * slim.h - C ABI of the SlimAttention / INT8 KV cache library for NVIDIA B200 (sm_100a).
 *
 * The library implements the attention hot path of "Inference Performance
 * Optimization for Large Language Models on CPUs" (arXiv 2407.07304):
 *   - Section 2.2: a KV cache stored as INT8 codes with one scale per token and
 *     per head, consumed by a hybrid-dtype kernel that converts the codes on the
 *     fly (there AVX-512 FMA; here tensor-core MMA);
 *   - Section 2.1: SlimAttention, a one-dimensional decomposition of attention:
 *     for a block of query rows the whole score row against all keys is formed,
 *     softmaxed once, and multiplied by V.
 * The paper does not fix the cache format; this library uses symmetric codes in
 * [-127, 127], scale = absmax / 127 stored as fp32, round half to even.
 *
 * General rules
 *   - Every pointer marked "device" must point to memory of the current CUDA
 *     device; pointers marked "host" are ordinary host memory.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream).  Unless stated otherwise no call synchronises
 *     with the host, allocates or frees memory, or keeps a pointer after it
 *     returns.
 *   - The caller owns every buffer.  The library never writes block_table or
 *     any length array.
 *   - Return value: SLIM_OK (0) or a negative SLIM_ERR_* code.  Arguments are
 *     validated on the host before anything is launched; a call that returns an
 *     error other than SLIM_ERR_CUDA has launched nothing.
 *   - Supported shapes: head_dim == 128, page_tokens == 128, Hq % Hkv == 0 and
 *     Hq / Hkv <= 16 for decode; Q and O are bf16.  Other shapes return
 *     SLIM_ERR_UNSUPPORTED.
 *   - Non-finite K/V/Q values are outside the contract.
 */
#ifndef SLIM_H_
#define SLIM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SLIM_OK               0
#define SLIM_ERR_INVALID_ARG (-1)  /* null pointer, negative size, inconsistent sizes */
#define SLIM_ERR_UNSUPPORTED (-2)  /* shape outside the supported set               */
#define SLIM_ERR_WORKSPACE   (-3)  /* workspace missing or too small                */
#define SLIM_ERR_CUDA        (-4)  /* a CUDA runtime call failed; see slim_last_cuda_error */
#define SLIM_ERR_TIMEOUT     (-5)  /* a bounded device-side wait ran out            */

#define SLIM_HEAD_DIM    128
#define SLIM_PAGE_TOKENS 128

#define SLIM_PHASE_PREFILL 0
#define SLIM_PHASE_DECODE  1

/*
 * Paged INT8 KV cache of one attention layer (Section 2.2).  A page holds
 * SLIM_PAGE_TOKENS consecutive token positions of one sequence, for every kv
 * head.  Token position `pos` of sequence b lives in page
 * block_table[b * max_pages_per_seq + pos / 128], slot pos % 128.
 *
 *   codes   device int8  [num_pages][num_kv_heads][2][128 slots][128 dims]   (index 0 = K, 1 = V)
 *   scales  device fp32  [num_pages][num_kv_heads][2][128 slots]
 *   block_table device int32 [B][max_pages_per_seq]; entries in [0, num_pages)
 *
 * A dequantised element is (float)code * scale of its (token, kv head).
 * codes and scales must be 16-byte aligned.  The struct itself is host memory
 * and is read during the call only.
 */
typedef struct slim_cache {
    int8_t        *codes;
    float         *scales;
    const int32_t *block_table;
    int32_t        num_pages;
    int32_t        page_tokens;        /* must be 128 */
    int32_t        num_kv_heads;
    int32_t        head_dim;           /* must be 128 */
    int32_t        max_pages_per_seq;
} slim_cache_t;

/*
 * Quantise new K and V rows and write them into the cache (Section 2.2: INT8
 * codes, one scale per (token, kv head), K and V separately).
 *
 * For each row x (128 bf16 values of one token and one kv head, K and V
 * separately): amax = max|x_d|; scale = amax / 127 (fp32, correctly rounded);
 * code_d = clamp(round_half_even(127 * x_d / amax), -127, 127); an all-zero row
 * gets scale 0 and codes 0.  Codes and scale bits are reproducible exactly.
 *
 *   k_new, v_new  device bf16 [total_new][num_kv_heads][128], the new tokens of
 *                 all sequences concatenated in sequence order; 16-byte aligned
 *   cu_new        device int32 [B+1]: rows cu_new[b] .. cu_new[b+1]-1 belong to
 *                 sequence b (cu_new[0] == 0)
 *   start_pos     device int32 [B]: cache position of sequence b's first new token
 *   B             number of sequences (>= 0; 0 is a no-op)
 *   max_new       upper bound on cu_new[b+1]-cu_new[b] (sizes the launch)
 *
 * The pages addressed through block_table must exist; a position past
 * max_pages_per_seq * 128 or a page id outside [0, num_pages) is skipped.
 */
int slim_kv_append(const slim_cache_t *cache, const void *k_new, const void *v_new,
                   const int32_t *cu_new, const int32_t *start_pos,
                   int32_t B, int32_t max_new, void *stream);

/*
 * Causal prefill attention over the INT8 cache (Section 2.1).  The new tokens'
 * K/V must already be in the cache (slim_kv_append first).
 *
 * This is the streamed form: a block of query rows owns every key it sees (the
 * one-dimensional decomposition of Section 2.1, no key split and no merge
 * between blocks), but 128-key tiles pass through the on-chip score buffer once,
 * behind a running row maximum, instead of the whole score row being formed
 * before its softmax.  The result is the same softmax attention; the order of
 * Section 2.1 itself is slim_attn_prefill_two_pass (any length) and
 * slim_attn_prefill_full_row (rows that see at most 256 keys).
 *
 * For sequence b with q_len = cu_q[b+1]-cu_q[b] query rows and kv_len[b] cached
 * tokens, query row t (0-based) sees keys j <= kv_len[b] - q_len + t; query
 * head h reads kv head h / (Hq / Hkv).  For each (row, head):
 *   s_j = sm_scale * sum_d q_d * (k_code[j][d] * k_scale[j]);  p = softmax_j(s);
 *   o_d = sum_j p_j * (v_code[j][d] * v_scale[j]).
 * A row that sees no key gets zeros.
 *
 *   q      device bf16 [total_q][Hq][128], 16-byte aligned
 *   out    device bf16 [total_q][Hq][128], 16-byte aligned
 *   cu_q   device int32 [B+1];   kv_len device int32 [B]
 *   max_q, max_kv  upper bounds on q_len and kv_len (size the launch)
 *   workspace      device scratch of at least
 *                  slim_workspace_bytes(SLIM_PHASE_PREFILL, ...) bytes (may be
 *                  NULL when that size is 0); its first 16 bytes are the status
 *                  word (see slim_read_status) and should be zero
 */
int slim_attn_prefill(const slim_cache_t *cache, const void *q, void *out,
                      const int32_t *cu_q, const int32_t *kv_len,
                      int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq, float sm_scale,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * The first-token phase in one call (Section 2.2: K and V are written to the
 * INT8 cache while the prompt is processed): exactly
 *   slim_kv_append(cache, k_new, v_new, cu_q, start_pos, B, max_q, stream) with
 *     start_pos[b] = kv_len[b] - (cu_q[b+1] - cu_q[b]), followed by
 *   slim_attn_prefill(cache, q, out, cu_q, kv_len, ...),
 * so kv_len[b] is the length of sequence b AFTER its new tokens, and every
 * query row has a new K / V row at the same index.  Two kernels; the second
 * is launched so that its set-up and its reads of q overlap the end of the
 * first (programmatic dependent launch), and the codes it reads are still in
 * the L2.  The rows are not quantised inside the attention kernel itself: a
 * key tile is read by every row block behind it (up to 64 at 16384 tokens),
 * each of which would have to quantise it again, or wait for the block that
 * owns it, which the longest-first order of the row blocks rules out.
 *
 *   k_new, v_new  device bf16 [total_q][num_kv_heads][128], 16-byte aligned
 *   other arguments, workspace and error behaviour as for slim_attn_prefill;
 *   codes and scales written are bit for bit those of slim_kv_append.
 */
int slim_prefill_step(const slim_cache_t *cache, const void *q, const void *k_new, const void *v_new, void *out,
                      const int32_t *cu_q, const int32_t *kv_len,
                      int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq, float sm_scale,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same attention in the literal order of Section 2.1: every score of a
 * query row is formed before its softmax.  The kernel walks a row block's keys
 * twice - first the row maxima of the scores, then P = exp(s - max) against
 * the final maximum and P.V - so no partial result is ever corrected.  It
 * forms Q.K^T twice and is therefore slower than slim_attn_prefill, which
 * streams the keys once behind a running maximum; it exists to measure that
 * difference.  Arguments, layout, workspace and error behaviour are those of
 * slim_attn_prefill; the two results agree within the output tolerance.
 */
int slim_attn_prefill_two_pass(const slim_cache_t *cache, const void *q, void *out,
                               const int32_t *cu_q, const int32_t *kv_len,
                               int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq, float sm_scale,
                               void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same attention with the whole score row on chip, the other literal form
 * of Section 2.1 (and the first row of the paper's Table 3, 256 tokens): for a
 * block of 128 query rows every score against all its keys is formed into one
 * strip of tensor memory, each row gets one softmax over its finished scores
 * (maximum, exponentials, sum - no running maximum, no second sweep over the
 * keys), and the strip is multiplied by V.  The strip is 128 rows x 256 fp32
 * scores beside the 128 x 128 output, which is what tensor memory holds: the
 * call serves caches of at most SLIM_FULL_ROW_MAX_KEYS tokens and returns
 * SLIM_ERR_UNSUPPORTED (nothing launched) when max_kv is larger; a kv_len[b]
 * beyond that limit attends over the first SLIM_FULL_ROW_MAX_KEYS tokens.
 * Arguments, layout, workspace and error behaviour otherwise as for
 * slim_attn_prefill; the results agree within the output tolerance.
 */
#define SLIM_FULL_ROW_MAX_KEYS 256
int slim_attn_prefill_full_row(const slim_cache_t *cache, const void *q, void *out,
                               const int32_t *cu_q, const int32_t *kv_len,
                               int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq, float sm_scale,
                               void *workspace, size_t workspace_bytes, void *stream);

/*
 * Decode attention: one query token per sequence against all kv_len[b] cached
 * tokens (the new token's K/V already appended).  Same arithmetic as above with
 * q_len == 1.  The next-token phase is a matrix-vector product bound by memory
 * bandwidth (Section 2.2, Eq. 1); the key range is split across thread blocks
 * and the pieces are merged by the log-sum-exp identity: by the split kernel
 * itself when its blocks finish where a row has few pieces, otherwise in a
 * second kernel.
 * A sequence with kv_len[b] == 0 gets zeros.
 *
 *   q, out   device bf16 [B][Hq][128], 16-byte aligned
 *   kv_len   device int32 [B];  max_kv upper bound on kv_len (sizes the launch)
 *   workspace device scratch of at least
 *             slim_workspace_bytes(SLIM_PHASE_DECODE, ...) bytes, 16-byte
 *             aligned.  Its first SLIM_WORKSPACE_HEADER_BYTES bytes (the status
 *             word, see slim_read_status, and the counters of the in-kernel
 *             merge) must be zero when the workspace is first used (one
 *             cudaMemset after allocating it); every call leaves the counters
 *             at zero again, so the same workspace serves any sequence of calls
 *             on one stream, whatever their shapes.  After a SLIM_ERR_TIMEOUT
 *             zero the header again.  The rest need not be initialised.
 */
#define SLIM_WORKSPACE_HEADER_BYTES (16 + 16384 * 4)
int slim_attn_decode(const slim_cache_t *cache, const void *q, void *out,
                     const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * The two passes of slim_attn_decode as separate calls, for callers that schedule
 * or time them individually: the split pass (every block: the scores of its key
 * chunk, one softmax over the chunk, the product with V; Section 2.1 order inside
 * the chunk) writes partials into `workspace`; the merge pass combines them into
 * `out`.  Same arguments, validation and workspace as slim_attn_decode, whose
 * result is that of split(..., NULL, NULL, ...) followed by merge(...) on the
 * same stream (where it merges inside the split kernel, up to the order of the
 * merge's sums).  With k_new and v_new (both or neither; as for
 * slim_decode_step) the split pass first writes every sequence's new token into
 * slot kv_len[b] - 1: slim_decode_step(...) computes split(..., k_new, v_new,
 * ...) followed by merge(...).
 */
int slim_attn_decode_split(const slim_cache_t *cache, const void *q, const void *k_new, const void *v_new,
                           const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                           void *workspace, size_t workspace_bytes, void *stream);
int slim_attn_decode_merge(const slim_cache_t *cache, void *out,
                           const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq,
                           const void *workspace, size_t workspace_bytes, void *stream);

/*
 * Decode attention with the keys of a sequence spread over several devices
 * (Section 2.3: the heads, and where there are fewer kv heads than devices the
 * key range, are split across workers and combined afterwards; in Eq. 1 the
 * batch, the heads and the tokens are plain factors).  Each device holds a
 * part of every sequence's tokens in a cache of its own (kv_len[b] = the tokens
 * it holds, possibly 0) and calls slim_attn_decode_partial, which is
 * slim_attn_decode without the final normalisation: for each (sequence, query
 * head) row it leaves the merged partial of the device's keys,
 *
 *   partial  device fp32 [B][Hq][SLIM_PARTIAL_FLOATS]: O[128] = sum_j 2^(s'_j - M) v^_j over the device's keys,
 *            then M (log2 units; -inf for a row without keys) and l = sum_j 2^(s'_j - M); 16-byte aligned.
 *
 * The devices exchange these rows (for 32 rows 17 KB per device) and every one
 * that needs the result calls slim_attn_merge_partials on the n_sets sets laid
 * out back to back: M = max M_r, l = sum l_r 2^(M_r - M),
 * o = sum O_r 2^(M_r - M) / l, written as bf16 [B][Hq][128].  The exchange itself
 * is the caller's (one all-gather); no kernel of this library reads another
 * device's memory.  Other arguments as for slim_attn_decode.
 */
#define SLIM_PARTIAL_FLOATS 132
int slim_attn_decode_partial(const slim_cache_t *cache, const void *q, float *partial,
                             const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                             void *workspace, size_t workspace_bytes, void *stream);
int slim_attn_merge_partials(const float *partials, int32_t n_sets, void *out, int32_t B, int32_t Hq, void *stream);

/*
 * One decode step in one call: the new token of every sequence is quantised into
 * the cache (exactly as slim_kv_append does, Section 2.2) at position
 * kv_len[b] - 1 and decode attention runs over all kv_len[b] tokens, the new one
 * included; the result equals slim_kv_append(start_pos = kv_len - 1) followed by
 * slim_attn_decode, bit for bit.  The quantisation happens inside the split
 * kernel of the attention (the thread block that reads a sequence's last key
 * chunk writes the new row first), so the step has no separate append kernel.
 *
 *   k_new, v_new  device bf16 [B][num_kv_heads][128], 16-byte aligned
 *   kv_len        device int32 [B]: cached tokens per sequence counting the new
 *                 one; a sequence with kv_len[b] <= 0 appends nothing and gets
 *                 zeros; a kv_len[b] beyond max_kv or the page table appends
 *                 nothing and attends over the tokens that fit
 *   others        as for slim_attn_decode
 */
int slim_decode_step(const slim_cache_t *cache, const void *q, const void *k_new, const void *v_new, void *out,
                     const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * One decode step from host buffers: brings the step's query and new K/V rows
 * (one new token per sequence) host -> device, runs slim_decode_step and brings
 * the result device -> host, all asynchronously on `stream` (Section 2.2: the
 * per-token step whose cache traffic Eq. 1 counts).  Host buffers should be pinned; they must stay
 * valid and unchanged, and out_host must not be read, until the stream has been synchronised.
 *
 * If the three input buffers are pinned memory that the device can address (cudaHostAlloc, cudaHostRegister)
 * and 16-byte aligned, the kernel reads them where they are - every row crosses the bus once, as in a copy, but
 * the step does not wait for a copy first.  Otherwise they are copied into `staging` (with one transfer instead
 * of three if q_host, k_new_host and v_new_host lie back to back in one allocation, in that order).  If out_host
 * is such pinned memory, the kernel writes the result straight into it and no copy back is issued; otherwise the
 * result goes through `staging` and a device -> host copy.
 *
 * The call synchronises nothing and allocates nothing.  After one ordinary call with the same cache and shapes
 * (which creates the tensor map and sets the kernels' attributes) it may be recorded by stream capture into a
 * CUDA graph; the graph reads the host buffers when it is replayed.
 *
 *   q_host      host bf16 [B][Hq][128]
 *   k_new_host, v_new_host  host bf16 [B][num_kv_heads][128]
 *   out_host    host bf16 [B][Hq][128]
 *   staging     device scratch of at least slim_step_staging_bytes(B, Hq, Hkv) bytes, 16-byte aligned
 *   kv_len      device int32 [B]: cached tokens per sequence counting the new one
 *   workspace   as for slim_attn_decode
 */
int slim_decode_step_host(const slim_cache_t *cache, const void *q_host, const void *k_new_host,
                          const void *v_new_host, void *out_host, void *staging, size_t staging_bytes,
                          const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                          void *workspace, size_t workspace_bytes, void *stream);
size_t slim_step_staging_bytes(int32_t B, int32_t Hq, int32_t Hkv);

/*
 * Decode attention for callers that cannot allocate device memory.  (The paper
 * has no counterpart to this call; it exists for integration reasons only.)
 *
 * Some hosts of this library are not allowed to call cudaMalloc at the point
 * where they run attention: code running while a CUDA graph is being captured,
 * a plug-in inside a serving runtime whose memory pool is owned and fully
 * reserved by someone else, or a real-time loop that must not take the
 * allocator's locks.  slim_attn_decode needs a workspace for the split pass's
 * partial results; this variant keeps those partials in a fixed array that is
 * part of the library image, so the caller passes inputs and outputs only.
 * It computes exactly what slim_attn_decode computes.
 *
 *  - The array is SLIM_STATIC_SCRATCH_BYTES (8 MiB) of device memory on every
 *    GPU that loads the library, held until the process exits.
 *  - A problem whose partials do not fit
 *    (slim_workspace_bytes(SLIM_PHASE_DECODE, ...) > SLIM_STATIC_SCRATCH_BYTES)
 *    is rejected with SLIM_ERR_WORKSPACE and nothing is launched; use
 *    slim_attn_decode with your own workspace for those.
 *  - No cudaMalloc/cudaFree and no allocating library routine is called.  The
 *    first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress, with that device current); make that first call
 *    before starting any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the last
 *    call left in it.  Its header starts at zero because the array is part of
 *    the zero-initialised image, and every call leaves it at zero; every other
 *    slot a call reads was written by that same call's split pass.  Two calls whose kernels
 *    can overlap on the GPU (different streams, no ordering between them) race
 *    on the array and give wrong results; keep calls on one stream or order
 *    them with events.
 *
 *  - The array's header (the status word of the bounded waits and the counters
 *    of the in-kernel merge) cannot be reached through slim_read_status or a
 *    memset, because the caller has no pointer to it.  slim_static_status does
 *    what slim_read_status does for a workspace (synchronises `stream`, returns
 *    SLIM_OK or SLIM_ERR_TIMEOUT); slim_static_reset enqueues a clear of the
 *    header on `stream` (one cudaMemsetAsync, nothing allocated) and must
 *    follow a SLIM_ERR_TIMEOUT before the next slim_attn_decode_static on that
 *    device, exactly as a workspace's header must be zeroed again: a kernel
 *    that gave up may have left counters non-zero, and later calls would then
 *    leave rows unwritten.  slim_static_selftest_timeout is
 *    slim_selftest_timeout aimed at the array's status word, so the sequence
 *    timeout -> status -> reset can be exercised without any fault.
 *  - The first of these four calls on a device performs the address lookup;
 *    host threads may make it concurrently.
 *
 * Arguments as for slim_attn_decode, minus the workspace.
 */
#define SLIM_STATIC_SCRATCH_BYTES (8 * 1024 * 1024)
int slim_attn_decode_static(const slim_cache_t *cache, const void *q, void *out,
                            const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                            void *stream);
int slim_static_status(void *stream);
int slim_static_reset(void *stream);
int slim_static_selftest_timeout(void *stream);

/*
 * Device-side waits are bounded.  The attention kernels wait on hardware barriers (TMA copies, tensor-core
 * completion); every such wait gives up after a fixed number of tries, and a kernel whose wait ran out
 * stores SLIM_ERR_TIMEOUT in the first word of its workspace and finishes with undefined output instead of
 * hanging.  slim_read_status synchronises `stream`, reads that word (host <- device) and returns SLIM_OK
 * or SLIM_ERR_TIMEOUT.  The kernels never clear the word: zero the header of a workspace once after
 * allocating it (16 bytes for prefill, SLIM_WORKSPACE_HEADER_BYTES for decode).
 */
int slim_read_status(const void *workspace, void *stream);

/*
 * Exercises that failure path without any failure: launches one thread that waits, with the kernels' bounded
 * wait and a short limit, on a barrier nothing arrives on; the wait runs out, the thread stores
 * SLIM_ERR_TIMEOUT in the first word of `workspace` (device, 4-byte aligned) and the kernel ends normally.
 * slim_read_status(workspace) then returns SLIM_ERR_TIMEOUT; the CUDA context stays usable.
 */
int slim_selftest_timeout(void *workspace, void *stream);

/* Scratch bytes needed by a phase (SLIM_PHASE_*) for the given shape; 0 on invalid arguments. */
size_t slim_workspace_bytes(int32_t phase, int32_t B, int32_t Hq, int32_t Hkv, int32_t max_q, int32_t max_kv);

/* Bytes of the codes and scales arrays of a pool of num_pages pages
 * (Eq. 1 with s_d = 1 for the codes, plus 2 fp32 scales per token and head). */
size_t slim_cache_code_bytes(int32_t num_pages, int32_t num_kv_heads);
size_t slim_cache_scale_bytes(int32_t num_pages, int32_t num_kv_heads);

/* Text for a return code; never NULL. */
const char *slim_strerror(int code);
/* The cudaError_t value behind the calling thread's last SLIM_ERR_CUDA (0 if none). */
int slim_last_cuda_error(void);
/* Library version, major * 10000 + minor * 100 + patch. */
int slim_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SLIM_H_ */

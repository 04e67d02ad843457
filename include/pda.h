/* pda.h -- C ABI of the B200 (sm_100a) paged decode attention library (libpda.so).
 *
 * One decode step of one attention layer over a paged KV cache:
 *
 *     kv_append  ->  paged_decode_attention  ( ->  paged_decode_reduce )
 *
 * The operation is the one the serving stacks of the paper run at every decode
 * step on top of their "paged KV cache" with grouped-query attention ("32 query
 * heads sharing 8 key/value heads", Appendix A, Scenario A): for sequence b and
 * query head h, with kv head g = h / (num_q_heads / num_kv_heads),
 *
 *     out[b,h,:] = softmax_j( scale * q[b,h,:] . K_j[g,:] ) . V_j[g,:]
 *
 * over the sequence's tokens j = 0 .. seq_lens[b]-1 in logical order, token j
 * living in physical page block_table[b][j / page_size], slot j % page_size.
 * The paper names these ingredients but defines no layout; everything below is
 * this library's definition.
 *
 * Conventions
 *   - All data pointers are DEVICE pointers unless a comment says "host".
 *   - The caller owns every data buffer: inputs, outputs, partials, workspaces,
 *     status words. TMA descriptors are rebuilt per call on the host and passed by
 *     value. What the library itself owns, per process, is small and listed here:
 *       * per device, a second stream and two events, created by the first
 *         paged_prefix_decode_attention call on that device that is not inside a
 *         stream capture (the cascade's suffix launch runs on it);
 *       * per device, 64 claim counters (256 bytes of the library's device image)
 *         used by the persistent kernel of paged_verify_attention, each left at zero
 *         by the launch that took it;
 *       * per device, the PDA_STATIC_SCRATCH_BYTES array of
 *         paged_decode_attention_static (part of the device image: reserved when the
 *         image is loaded on that device, see there);
 *       * one host-side integer, the threshold of pda_set_persistent_threshold.
 *     No call allocates device memory with cudaMalloc or frees any; nothing else
 *     is kept between calls.
 *   - Every call enqueues work on `stream` (a cudaStream_t passed as void*) and
 *     returns without synchronising. Nothing reads seq_lens or block_table back
 *     to the host, so a step can be captured in a CUDA graph.
 *   - Return value: 0 = PDA_OK; < 0 = PDA_ERR_* detected on the host before
 *     anything was enqueued; > 0 = the cudaError_t of a failed launch.
 *   - `status` (optional, device int32, caller-zeroed): problems found on the
 *     device are recorded with atomicMax(status, PDA_DEV_*). The affected unit's
 *     output is zero-filled; no out-of-bounds access is ever made.
 *   - bf16 = upper half of an IEEE binary32. e4m3 = OCP FP8 E4M3 (bias 7, max
 *     finite 448, no infinities, S.1111.111 = NaN).
 */
#ifndef PDA_H_
#define PDA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PDA_VERSION 100

/* host-side return codes */
#define PDA_OK 0
#define PDA_ERR_INVALID_ARG (-1)  /* null pointer, negative size, inconsistent sizes          */
#define PDA_ERR_UNSUPPORTED (-2)  /* shape / dtype / stride outside the supported set          */
#define PDA_ERR_MISALIGNED (-3)   /* a pointer or stride breaks the 16-byte alignment rule     */
#define PDA_ERR_TOO_LARGE (-4)    /* size beyond a documented fixed maximum                    */

/* device-side status codes (atomicMax into *status) */
#define PDA_DEV_OK 0
#define PDA_DEV_BAD_PAGE 1     /* block_table entry outside [0, num_pages) for a live page     */
#define PDA_DEV_BAD_SEQ_LEN 2  /* seq_lens[b] > block_table_stride * page_size                 */
#define PDA_DEV_TIMEOUT 3      /* a bounded wait on an asynchronous copy expired               */

/* KV element types */
#define PDA_BF16 0
#define PDA_FP8_E4M3 1

/* flags for paged_decode_attention */
#define PDA_FLAG_FORCE_GENERIC 1u /* use the plain CUDA-core kernel even where the
                                     TMA + tensor-core kernel applies (for testing) */

#define PDA_FLAG_MQ_MMA_SYNC 2u   /* multi-query calls (verify, shared prefix): use the mma.sync
                                     kernel even where the tcgen05 + TMEM kernel applies */
#define PDA_FLAG_MQ_ONE_UNIT 4u   /* paged_verify_attention: one CTA per (sequence, kv head, row block) even
                                     where a persistent tcgen05 kernel applies (unsplit, head_dim 128) */

typedef void* pda_stream_t; /* cudaStream_t */

/* Describes k_cache and v_cache (both have the same geometry).
 * Element (page, head, slot, d) lives at element offset
 *   page*page_stride + head*head_stride + slot*slot_stride + d.
 * The canonical layout is [num_pages, num_kv_heads, page_size, head_dim]
 * contiguous, i.e. slot_stride = head_dim, head_stride = page_size*head_dim,
 * page_stride = num_kv_heads*head_stride; any strides whose byte values are
 * multiples of 16 are accepted. */
typedef struct pda_cache_desc {
  int64_t page_stride;  /* elements */
  int64_t head_stride;  /* elements */
  int64_t slot_stride;  /* elements */
  int32_t num_pages;
  int32_t page_size;    /* tokens per page; supported: 16 */
  int32_t num_kv_heads;
  int32_t head_dim;     /* supported: multiples of 32 up to 256; fast path 64 and 128 */
  int32_t dtype;        /* PDA_BF16 or PDA_FP8_E4M3 */
} pda_cache_desc;

int pda_version(void);
const char* pda_status_string(int code); /* text for a PDA_ERR_* / PDA_DEV_* / 0 code */

/* ceil(max_seq_len / chunk_tokens): the `max_chunks` extent the partial buffers need. */
int pda_max_chunks(int32_t max_seq_len, int32_t chunk_tokens);

/* KV append (this step's scatter of new keys/values into the paged cache; the
 * paper's Appendix A lists the paged KV cache, not its update rule -- this is
 * the plain definition): for every sequence b with L = seq_lens[b] > 0 (length
 * AFTER the append) and every kv head g,
 *     cache[block_table[b][(L-1)/P]][g][(L-1)%P][:] = new[b][g][:]   (bytewise)
 * k_new, v_new: [batch, num_kv_heads, head_dim] bf16, contiguous. bf16 caches
 * only (PDA_ERR_UNSUPPORTED for e4m3). Target slots must be distinct across the
 * batch. A bad page id or length skips that sequence and sets *status.
 * desc is a host pointer, read during the call. */
int kv_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
              const pda_cache_desc* desc, const int32_t* block_table,
              int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
              int32_t* status, pda_stream_t stream);

/* Paged decode attention (definition at the top of this file; GQA head grouping
 * per Appendix A, Scenario A).
 *   q            [batch, num_q_heads, head_dim] bf16, contiguous
 *   k_scale,
 *   v_scale      [num_pages, num_kv_heads] fp32 dequantisation factors for e4m3
 *                caches (value = decode(byte) * scale); NULL for bf16 caches
 *   block_table  [batch, block_table_stride] int32; entries at or beyond
 *                ceil(seq_lens[b]/page_size) are never read
 *   scale        fp32 multiplier of q.k
 *   chunk_tokens 0: whole sequence per unit, result written to `out`
 *                [batch, num_q_heads, head_dim] bf16 (round to nearest even);
 *                a sequence of length 0 gives zeros.
 *                >0 (multiple of page_size): split-KV. Chunk c covers tokens
 *                [c*chunk_tokens, min((c+1)*chunk_tokens, L)); for every c <
 *                ceil(L/chunk_tokens) the kernel writes
 *                  part_o  [batch, num_q_heads, max_chunks, head_dim] fp32,
 *                          normalised within the chunk, and
 *                  part_lse[batch, num_q_heads, max_chunks] fp32 = m + ln(l)
 *                          (natural log of the chunk's softmax denominator);
 *                other entries are left untouched; `out` is not written.
 *                max_chunks * chunk_tokens must cover block_table_stride*page_size
 *                or at least every seq_lens[b] (longer sequences set *status).
 *   flags        PDA_FLAG_* bits
 * Unused slots of a last page, unused pages and table tails may hold any bit
 * pattern (NaN included). e4m3 caches: q is converted to fp16 for the tensor
 * core path, so |q| must stay below 65504.
 * Supported: page_size 16; num_q_heads a multiple of num_kv_heads; any group
 * size and head_dim (multiple of 32, <= 256) on the generic kernel; group size
 * <= 8 with head_dim 64 or 128 on the TMA + tensor-core kernel. */
int paged_decode_attention(const void* q, const void* k_cache, const void* v_cache,
                           const pda_cache_desc* desc, const float* k_scale,
                           const float* v_scale, const int32_t* block_table,
                           int32_t block_table_stride, const int32_t* seq_lens,
                           int32_t batch, int32_t num_q_heads, float scale,
                           int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                           int32_t max_chunks, uint32_t flags, int32_t* status,
                           pda_stream_t stream);

/* Sliding-window decode attention: paged_decode_attention restricted, for every
 * sequence, to its last `window` tokens j in [max(0, L - window), L) (the
 * sliding-window attention over a paged per-stream cache of the paper's
 * streaming scenario, Appendix A, Scenario D; the paper gives no formula -- this
 * is the same softmax over that token range). window == 0 means no window.
 * Pages wholly before the window are never read, so their block_table entries
 * may be stale (evicted pages). With chunk_tokens > 0 the chunk grid stays the
 * one of the full sequence: chunks wholly before the window get o = 0 and
 * lse = -inf, and paged_decode_reduce merges as usual. Other arguments as in
 * paged_decode_attention. */
int paged_window_decode_attention(const void* q, const void* k_cache, const void* v_cache,
                                  const pda_cache_desc* desc, const float* k_scale,
                                  const float* v_scale, const int32_t* block_table,
                                  int32_t block_table_stride, const int32_t* seq_lens,
                                  int32_t batch, int32_t num_q_heads, float scale, int32_t window,
                                  int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                                  int32_t max_chunks, uint32_t flags, int32_t* status,
                                  pda_stream_t stream);

/* Append of n_new tokens per sequence (the draft block of a verification step):
 * k_new, v_new are [batch, n_new, num_kv_heads, head_dim] bf16; token i becomes
 * logical token seq_lens[b] - n_new + i (seq_lens = length AFTER the append).
 * n_new == 1 is kv_append. */
int kv_append_tokens(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                     const pda_cache_desc* desc, const int32_t* block_table,
                     int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                     int32_t n_new, int32_t* status, pda_stream_t stream);

/* Quantising KV append into e4m3 caches (no counterpart in the paper, whose one
 * remark on KV quantisation is negative; this is the library's policy). k_new,
 * v_new: [batch, num_kv_heads, head_dim] bf16. For K and V separately and every kv
 * head, with slot = (L-1) % page_size of the target page:
 *   slot == 0: scale[page, head] = amax(row) * 2 / 448 (1 if the row is all zero)
 *              is stored -- the page's scale is fixed by its first row;
 *   slot  > 0: the stored scale is reused;
 *   bytes = e4m3(row / scale): IEEE fp32 division, round to nearest even,
 *           saturating at +-448.
 * k_scale, v_scale: [num_pages, num_kv_heads] fp32, read and written. head_dim must
 * be a multiple of 64. Target slots must be distinct across the batch. */
int kv_append_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                  const pda_cache_desc* desc, float* k_scale, float* v_scale,
                  const int32_t* block_table, int32_t block_table_stride,
                  const int32_t* seq_lens, int32_t batch, int32_t* status, pda_stream_t stream);

/* The same for a block of n_new tokens per sequence (the draft block of a
 * verification step on an e4m3 cache): k_new, v_new are
 * [batch, n_new, num_kv_heads, head_dim] bf16, token i becomes logical token
 * seq_lens[b] - n_new + i, and the one-token rule above is applied to the tokens
 * in this order -- a page opened inside the block takes its scale from the
 * block's own row that lands in its slot 0. n_new == 1 is kv_append_fp8. */
int kv_append_tokens_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                         const pda_cache_desc* desc, float* k_scale, float* v_scale,
                         const int32_t* block_table, int32_t block_table_stride,
                         const int32_t* seq_lens, int32_t batch, int32_t n_new, int32_t* status,
                         pda_stream_t stream);

/* Verification attention over a block of n_query_tokens draft tokens per sequence
 * (the predicted-output verifier of the paper scores 16-token blocks in one pass:
 * Section 4.2 and Appendix A, Scenario B; the paper prints no formula -- this is
 * causal attention over the paged cache). The cache already holds all seq_lens[b]
 * tokens, the block being the last n_query_tokens of them; query token i stands at
 * position L - n + i and attends tokens j <= L - n + i.
 *   q, out    [batch, n_query_tokens, num_q_heads, head_dim] bf16
 *   chunk_tokens 0: one unit per (sequence, kv head).  > 0: split-KV; the partials
 *             part_o [batch, n, num_q_heads, max_chunks, head_dim] and part_lse
 *             [batch, n, num_q_heads, max_chunks] are scratch and the merge runs
 *             inside this call.  `out` is always written.
 * The query rows of a kv head's group form dense tensor-core tiles (rows = tokens x
 * group size), so each page is fetched once per block, not once per token.
 * bf16 KV with head_dim 128 or 64 and e4m3 KV with head_dim 128 run on tcgen05
 * tensor-core tiles with the accumulators in tensor memory (128 query rows per CTA);
 * PDA_FLAG_MQ_MMA_SYNC selects the mma.sync kernel instead. Unsplit calls with
 * head_dim 128 and up to 1024 sequences run as one persistent CTA per SM that walks
 * through the (sequence, kv head, row block) units, longest sequences first
 * (PDA_FLAG_MQ_ONE_UNIT: one CTA per unit). The bf16 one of these kernels shares out its last
 * units through a counter in device memory which the library owns (a pool of 64,
 * taken in turn by the launches and left at zero by each): up to 64 such launches
 * may be in flight at once on a device; a launch captured in a CUDA graph keeps its
 * counter, so one graph must not run beside itself on two streams.
 * e4m3 on tcgen05: the products are e4m3 x e4m3 on the cache's bytes; q enters as two
 * e4m3 parts (exact for every element within 2^-9 of its row's largest) and the softmax
 * weights as three 8-bit parts that add up to the weight rounded to fp16, the same
 * precision the mma.sync kernel gives them; the page scales go through the softmax.
 * Scales must be finite and non-negative (kv_append_fp8 writes them so). */
int paged_verify_attention(const void* q, const void* k_cache, const void* v_cache,
                           const pda_cache_desc* desc, const float* k_scale,
                           const float* v_scale, const int32_t* block_table,
                           int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                           int32_t num_q_heads, int32_t n_query_tokens, float scale,
                           int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                           int32_t max_chunks, uint32_t flags, int32_t* status,
                           pda_stream_t stream);

/* Decode attention for a batch whose sequences all start with the SAME
 * prefix_tokens tokens stored in the same physical pages (the shared-prefix
 * prompt-caching workload of the paper: Section 4.2 and Appendix A, Scenario C).
 * The result is exactly paged_decode_attention's; the work is reorganised: the
 * prefix's keys/values are read once for the whole batch (all queries of a kv
 * head's groups as one block of rows), each sequence's own suffix is attended
 * separately, and the pieces are merged by their log-sum-exp weights.
 *   block_table    rows must agree on their first prefix_tokens/page_size entries
 *                  (row 0's are used); prefix_tokens is a multiple of page_size and
 *                  <= every seq_lens[b]
 *   prefix_chunk_tokens  split of the prefix for parallelism (multiple of page_size). The
 *                  prefix launch has ceil(batch * group / 128) * num_kv_heads CTAs per chunk,
 *                  each with a fixed cost of several microseconds: fastest with at most one
 *                  CTA per SM and chunks of 1024 tokens or more
 *   chunk_tokens   (> 0) split of the suffixes
 *   part_o, part_lse  scratch [batch, num_q_heads, max_chunks, head_dim] / [.., max_chunks]
 *                  with max_chunks >= ceil(prefix_tokens/prefix_chunk_tokens)
 *                                    + ceil((max seq_len - prefix_tokens)/chunk_tokens)
 *   out            [batch, num_q_heads, head_dim] bf16
 * Three launches (prefix, suffixes, merge), ordered on `stream`; the suffix launch,
 * which is independent of the prefix launch, runs beside it on a stream the
 * library owns (forked from and joined back to `stream` with events, which is
 * also valid while `stream` is being captured; the side stream is created by the
 * first call that is not inside a capture, and until it exists the launches simply
 * follow one another on `stream`). Supported: group size <= 8, head_dim 64/128
 * (bf16) or 128 (e4m3), batch <= 4096. The prefix launch is a multi-query call:
 * the kernel choice, `flags` and the e4m3 precision note of paged_verify_attention
 * apply to it. */
int paged_prefix_decode_attention(const void* q, const void* k_cache, const void* v_cache,
                                  const pda_cache_desc* desc, const float* k_scale,
                                  const float* v_scale, const int32_t* block_table,
                                  int32_t block_table_stride, const int32_t* seq_lens,
                                  int32_t batch, int32_t num_q_heads, float scale,
                                  int32_t prefix_tokens, int32_t prefix_chunk_tokens,
                                  int32_t chunk_tokens, void* out, float* part_o, float* part_lse,
                                  int32_t max_chunks, uint32_t flags, int32_t* status,
                                  pda_stream_t stream);

/* Merge of split-KV partials (the reduce step of flash-decoding; exact algebra):
 *     out[b,h,:] = sum_c w_c part_o[b,h,c,:] / sum_c w_c,
 *     w_c = exp(part_lse[b,h,c] - max_c part_lse[b,h,c]),  c < ceil(L_b/chunk_tokens)
 * out: [batch, num_q_heads, head_dim] bf16. A sequence without chunks gives zeros. */
int paged_decode_reduce(const float* part_o, const float* part_lse, const int32_t* seq_lens,
                        int32_t batch, int32_t num_q_heads, int32_t head_dim,
                        int32_t chunk_tokens, int32_t max_chunks, void* out,
                        pda_stream_t stream);

/* Tuning knob (process-wide, host side): an unsplit paged_decode_step with a workspace
 * and batch <= 256 runs on the persistent kernel (resident CTAs looping over (sequence, kv
 * head) units through the workspace's work ticket, longest first) once there are at least
 * min_units_per_cta units per resident CTA (2 per SM); below that, one CTA per unit is
 * faster. Default 6. 0 always selects the persistent kernel where it applies (tests). */
int pda_set_persistent_threshold(int32_t min_units_per_cta);

/* Number of int32 the `workspace` of paged_decode_step needs: 2 + batch*num_kv_heads. */
int pda_workspace_ints(int32_t batch, int32_t num_kv_heads);

/* One whole decode step of this layer in a single launch: KV append (when k_new
 * and v_new are given; both NULL skips it), paged decode attention and, for
 * chunk_tokens > 0, the merge of the split-KV partials -- the three calls above
 * fused, with the same definitions; `out` [batch, num_q_heads, head_dim] bf16 is
 * always written. The append is applied to the cache and seen by this step's
 * attention.
 *   part_o, part_lse, max_chunks  as in paged_decode_attention (chunk_tokens > 0)
 *   workspace  device int32[pda_workspace_ints(batch, num_kv_heads)], zeroed by the
 *              caller ONCE (e.g. at allocation); every call leaves it zeroed again,
 *              so consecutive calls on one stream may share it. Calls that can
 *              overlap on the GPU need separate workspaces. It carries the work
 *              the work ticket of the persistent kernel (two leading ints)
 *              and the per-(sequence, kv head) chunk counters. May be NULL when chunk_tokens == 0. After a
 *              PDA_DEV_TIMEOUT status, zero it again.
 * If chunk_tokens > 0 and workspace is NULL, or the shape is outside the fused
 * kernel's set (group size > 8, head_dim not 64/128), the step is
 * run as the separate launches instead, with the same result. */
int paged_decode_step(const void* q, const void* k_new, const void* v_new, void* k_cache,
                      void* v_cache, const pda_cache_desc* desc, const float* k_scale,
                      const float* v_scale, const int32_t* block_table,
                      int32_t block_table_stride, const int32_t* seq_lens, int32_t batch,
                      int32_t num_q_heads, float scale, int32_t chunk_tokens, void* out,
                      float* part_o, float* part_lse, int32_t max_chunks, int32_t* workspace,
                      int32_t* status, pda_stream_t stream);

/* seq_lens[b] += delta for every b, on the device and in stream order. Lets a
 * whole decode step -- advance the lengths, then paged_decode_step -- be captured
 * once in a CUDA graph and replayed every token with no host work (CUDA-graph
 * capture of the step is the most frequent single win the paper reports:
 * Section 4.2, Scenarios B, C, D and F). Grids never depend on seq_lens, the
 * caches' addresses are baked into the captured launch, and the block table must
 * already hold the pages the growing sequences will reach. */
int pda_advance_seq_lens(int32_t* seq_lens, int32_t batch, int32_t delta, pda_stream_t stream);

/* One whole decode step driven from HOST buffers (the end-to-end call): copies
 * this step's q, k_new, v_new, seq_lens and block_table from (ideally pinned)
 * host memory into the caller's device staging buffers, runs
 * paged_decode_step (workspace as described there, may be NULL), and copies
 * `out` back to out_host; all on `stream`, without synchronising. The KV cache
 * itself stays resident on the device between steps. *_dev are device buffers
 * of the same sizes as their host counterparts.
 * In place: q_dev, k_new_dev, v_new_dev, block_table_dev, seq_lens_dev and
 * out_dev may each be NULL; the kernel then reads (for out: writes) the host
 * buffer itself over the bus while it streams the cache, and that copy and its
 * launch drop out of the step. This needs pinned host memory that is mapped into
 * the device's address space (cudaHostAlloc, cudaHostRegister);
 * PDA_ERR_INVALID_ARG otherwise. With out_dev == NULL the result exists in
 * out_host only. Every CTA reads seq_lens and its row of block_table at its
 * start, so reading those two in place trades two copies ahead of the launch
 * for a bus round trip inside each CTA's start; the host must not change any
 * in-place buffer before the step has completed. */
int paged_decode_step_host(const void* q_host, const void* k_new_host, const void* v_new_host,
                           const int32_t* block_table_host, const int32_t* seq_lens_host,
                           void* q_dev, void* k_new_dev, void* v_new_dev,
                           int32_t* block_table_dev, int32_t* seq_lens_dev,
                           void* k_cache, void* v_cache, const pda_cache_desc* desc,
                           int32_t block_table_stride, int32_t batch, int32_t num_q_heads,
                           float scale, int32_t chunk_tokens, float* part_o, float* part_lse,
                           int32_t max_chunks, int32_t* workspace, void* out_dev, void* out_host,
                           int32_t* status, pda_stream_t stream);

/* Split-KV attention plus reduce with library-owned scratch. (The paper has no
 * counterpart; this entry point exists for integration reasons only.)
 *
 * Some callers cannot hand the library partial buffers because they cannot get
 * device memory when the call is made: a serving process whose start-up code has
 * already claimed the whole HBM for its KV pool and weights, so that any later
 * cudaMalloc fails; a plug-in that runs inside a host application's context and
 * was given no allocator; or a latency-critical loop in which an allocation's
 * implicit device synchronisation is not acceptable. For them this call does what
 * paged_decode_attention(chunk_tokens > 0) followed by paged_decode_reduce does,
 * but keeps part_o / part_lse in a fixed array of PDA_STATIC_SCRATCH_BYTES
 * compiled into the library's device image. It calls no cudaMalloc, cudaFree or
 * other allocating routine.
 *
 * The array is part of the device code of the library, and the CUDA runtime loads
 * device code lazily: the image that holds the array is loaded on a device -- and
 * its PDA_STATIC_SCRATCH_BYTES of device memory reserved there, until the process
 * exits -- by the FIRST call of this function on that device, which looks up the
 * array's device address (with that device current) and caches it. That first
 * call therefore synchronises like any module load and fails with the runtime's
 * out-of-memory code (a positive return value) if the device has no room left.
 * Make it once per device at start-up: before the process hands the rest of HBM
 * to its pools, and outside any stream capture (a call with batch 0 is enough and
 * enqueues nothing). Every later call on that device reserves nothing: the free
 * memory the runtime reports is the same before and after it.
 *
 * Arguments are those of paged_decode_attention without the partial buffers and
 * flags; `out` is [batch, num_q_heads, head_dim] bf16. The sizes must satisfy
 *   round_up(batch*num_q_heads*max_chunks*head_dim*4, 256)
 *     + batch*num_q_heads*max_chunks*4  <=  PDA_STATIC_SCRATCH_BYTES,
 * otherwise PDA_ERR_TOO_LARGE is returned and nothing is enqueued.
 *
 * The array is shared by all calls and keeps the previous call's contents:
 * nothing in it needs to start at zero (attention writes every entry that reduce
 * reads), but two calls whose kernels can overlap on the GPU (different streams,
 * or different host threads without ordering) race on it. Calls on one stream are
 * ordered and safe. */
#define PDA_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
int paged_decode_attention_static(const void* q, const void* k_cache, const void* v_cache,
                                  const pda_cache_desc* desc, const float* k_scale,
                                  const float* v_scale, const int32_t* block_table,
                                  int32_t block_table_stride, const int32_t* seq_lens,
                                  int32_t batch, int32_t num_q_heads, float scale,
                                  int32_t chunk_tokens, int32_t max_chunks, void* out,
                                  int32_t* status, pda_stream_t stream);

/* Diagnostic: decodes all 256 e4m3 bytes with the device decoder the generic
 * kernel uses; out256: device float[256]. */
int pda_debug_e4m3_decode(float* out256, pda_stream_t stream);

/* Diagnostic: makes the kernels' bounded waits run out. (No counterpart in the
 * paper; this exercises the library's own failure handling.) Every wait inside the
 * attention kernels is a wait of a warp on an mbarrier of its own CTA with a poll
 * limit, after which the kernel records PDA_DEV_TIMEOUT in *status, zero-fills the
 * unit's output and returns. This call launches one warp that initialises such a
 * barrier, never arrives at it, and runs the same two wait helpers (the suspended
 * try_wait form of the TMA rings, the spinning test_wait form of the tensor-core
 * hand-offs) with `polls` as their limit instead of the built-in 2^18 (4.0 us per
 * poll: 1.05 s) and 2^24 (21.9 ns per poll: 0.37 s).
 * Nothing faults and nothing waits without a limit; the context stays usable.
 *   polls   1 .. 2^20
 *   status  device int32: receives atomicMax(PDA_DEV_TIMEOUT)
 *   result  device uint64[3] or NULL: nanoseconds spent in the suspended and in the
 *           spinning wait, and a mask of the waits that wrongly reported completion
 *           (must be 0). */
int pda_debug_wait_timeout(uint32_t polls, int32_t* status, uint64_t* result, pda_stream_t stream);

/* Diagnostic: read-only streaming probe. Reads `bytes` (a multiple of 16) from the
 * 16-byte aligned device buffer `buf` once with 16-byte loads from 8 CTAs per SM
 * and writes nothing but (practically never) one counter word `sink` (device
 * uint32). Timed by the caller with events, bytes / time is the bandwidth a kernel
 * that only reads HBM can reach on this device: the ceiling beside which the
 * decode kernels' GB/s are to be read (a copy moves half its bytes as writes and
 * is the lower figure). */
int pda_debug_read_probe(const void* buf, uint64_t bytes, uint32_t* sink, pda_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* PDA_H_ */

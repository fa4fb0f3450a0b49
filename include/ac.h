/*
 * ac.h -- C ABI of the B200 (sm_100a) paged decode-attention library (libac.so).
 *
 * One decode step of one attention layer, for a batch of requests that each contribute ONE new
 * token, over a paged KV cache:
 *
 *   ac_rope_kv_append      rotary embedding of the new q and k, then the new k/v are written into
 *                          their cache page through the block table
 *   ac_paged_decode_attn   grouped-query attention of each request's query token over all of its
 *                          cached pages, one CTA per (request, KV head, KV split), online softmax;
 *                          emits per-split partial results (or the final output when 1 split)
 *   ac_splitkv_merge       log-sum-exp merge of the per-split partial results
 *
 * Source of each operation (the paper gives them in prose only): Method, "Principle-Driven LLM
 * Kernel Generator", kernel families (iii) "standalone RoPE kernel" and (iv) "paged decode
 * attention ... online-softmax kernel over paged KV with fused cross-CTA merging"; Method, "Kernel
 * Customization and Multi-Request Adaptation": the kv_append scatter kernel ("writes the new K/V
 * vectors", attention then runs "with the sequence length advanced by one"), the paged KV cache
 * allocated at block granularity, sequence lengths kept on the GPU, and decode steps replayed as
 * bucketed CUDA Graphs (one graph per batch-size bucket).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer owned by the caller unless its name ends in _host or
 *     _out.  The library never allocates or frees device memory, never synchronises and never reads
 *     device memory on the host: each call only validates its arguments and enqueues work on
 *     `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).  The three kernel
 *     calls may therefore be recorded in a CUDA Graph; ac_init must have been called before capture.
 *   - The kernels are launched with programmatic stream serialization and signal launch completion
 *     early, so that in a chain of calls each kernel's set-up overlaps the tail of the one before.
 *     Before synchronising on the preceding kernel the attention kernels read only context_lens,
 *     block_table and cache tiles below the one holding slot context_lens[b] - 1, and the projection
 *     kernels only their weights.  The attention and RoPE kernels signal only after their own
 *     synchronisation, so no kernel that writes the cache can still be running two launches back:
 *     consecutive steps on one cache need nothing between them.  The early reads are invisible
 *     unless the kernel enqueued directly before one of these calls BOTH writes context_lens,
 *     block_table or those weights AND itself signals programmatic launch completion before
 *     finishing; such a producer must not signal early (copies and ordinary kernels are always safe).
 *   - Tensors q/k/v/cache/out are bf16 (16-bit patterns); rope tables and partials are fp32;
 *     block_table and context_lens are int32.  The innermost dimension (head_dim) is contiguous.
 *   - Return value: AC_OK (0) or an ac_status > 0.  On any non-zero return nothing was launched.
 *     The library never throws, aborts or exits.
 *   - Supported: head_dim d in {64, 128}; page_size a multiple of 16, <= 256; Hq % Hkv == 0 and
 *     Hq / Hkv <= 16; all base pointers 16-byte aligned; cache strides multiples of 8 elements and
 *     stride_token, stride_head >= d.
 *   - Rows with context_lens[b] < 0 are inactive (batch padding up to a graph bucket): nothing is
 *     written to the cache for them and their output row is +0.
 *   - Query head hq reads KV head hq / (Hq / Hkv).
 */
#ifndef AC_H_
#define AC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AC_OK = 0,
    AC_ERR_NULL = 1,        /* a required pointer is NULL */
    AC_ERR_SHAPE = 2,       /* a size is non-positive or inconsistent */
    AC_ERR_UNSUPPORTED = 3, /* outside the supported set listed above */
    AC_ERR_ALIGN = 4,       /* pointer or stride alignment */
    AC_ERR_WORKSPACE = 5,   /* workspace too small for num_splits */
    AC_ERR_CUDA = 6,        /* a CUDA call failed; see ac_last_cuda_error() */
    AC_ERR_NOT_INIT = 7,    /* ac_init has not succeeded on the current device */
    AC_ERR_SCRATCH_LIMIT = 8 /* ac_paged_decode_attn_static_scratch: partials exceed AC_STATIC_SCRATCH_BYTES */
} ac_status;

/* Bits the kernels OR into the optional device word `status_flag` (never cleared by the library). */
#define AC_FLAG_PAGE_OOB 1     /* a block-table entry used for the append was outside [0, num_pages) */
#define AC_FLAG_POSITION_OOB 2 /* context_lens[b] >= max_position or its page index >= max_pages_per_seq; in the
                                  single-launch step also context_lens[b] + 1 > the tokens the split grid covers */
#define AC_FLAG_WAIT_TIMEOUT 4 /* a bounded wait on a shared-memory barrier gave up */

/* Once per device, outside any stream capture, with no other call of this library running on that
 * device: reads the device properties, resolves the driver's tensor-map encoder and sets the
 * dynamic shared-memory limits of every kernel instantiation.  device < 0 means the current device.
 * Idempotent. */
int ac_init(int device);

/* Static, never-freed description of a status code. */
const char* ac_status_string(int status);

/* cudaError_t (or CUresult, for tensor-map encoding) recorded by the last AC_ERR_CUDA on this thread. */
int ac_last_cuda_error(void);

/* Number of SMs of the device ac_init saw last; 0 before any ac_init. */
int ac_sm_count(void);

/* Split plan (host only, pure, needs no GPU).  Chooses how many KV splits the attention kernel
 * should use for `sm_count` SMs (<= 0: the count seen by ac_init, or 148 if none): none when the
 * (request, KV head) pairs alone fill the GPU and contexts are short, chunks of at most 4096 tokens
 * when contexts are long, and otherwise the split count with the smallest estimated time from a
 * small cost model (bandwidth of one CTA, waves of CTAs, partial-result traffic); splits are never
 * shorter than 256 tokens, or 128 where the grid is small enough for the merge inside a cluster.  max_context_len = the largest number of tokens any row attends over in this bucket
 * (cached + new).  Outputs: *num_splits_out >= 1, *split_tokens_out = tokens per split (a multiple
 * of 64; split s of row b covers tokens [s*split_tokens, min((s+1)*split_tokens, n_b)) ), and
 * *workspace_bytes_out = bytes of fp32 workspace the attention + merge calls need for that plan
 * (0 when num_splits == 1).  The paper's kernel merges across CTAs inside the attention kernel and
 * does not state how it sizes the split; this heuristic is this library's own. */
int ac_decode_plan(int B, int Hq, int Hkv, int d, int page_size, int max_context_len, int sm_count,
                   int* num_splits_out, int* split_tokens_out, size_t* workspace_bytes_out);

/* The same plan for a batch whose row lengths the caller knows (a scheduler builds context_lens on
 * the host anyway).  token_counts_host[b] = tokens row b attends over this step (cached + new; <= 0
 * for an inactive row), a HOST array of B entries; max_context_len >= every entry bounds the chunk
 * grid as in ac_decode_plan (counts above it are clipped).  Splits that lie beyond a row's end launch
 * CTAs that exit at once, so a ragged batch can afford more and shorter splits than its longest row
 * alone suggests: the estimate counts only the CTAs that have tokens, the longest of them, and the
 * batch's total bytes.  Same outputs and errors as ac_decode_plan; any plan gives the same results. */
int ac_decode_plan_for_lengths(const int32_t* token_counts_host, int B, int Hq, int Hkv, int d,
                               int page_size, int max_context_len, int sm_count,
                               int* num_splits_out, int* split_tokens_out, size_t* workspace_bytes_out);

/* Tokens per split the attention kernel uses for a given (max_context_len, num_splits): the smallest
 * multiple of 64 whose num_splits-fold covers max_context_len.  Host only, pure. */
int ac_split_tokens(int max_context_len, int num_splits);

/* Workspace bytes for (B, Hq, d, num_splits): partial_o fp32 [B,Hq,num_splits,d] followed by
 * partial_lse fp32 [B,Hq,num_splits]; 0 when num_splits == 1.  Host only, pure. */
size_t ac_workspace_bytes(int B, int Hq, int d, int num_splits);

/* A1 + A2: RoPE on the new q/k and KV append (families (iii) "standalone RoPE kernel" and the
 * kv_append scatter kernel of "Kernel Customization and Multi-Request Adaptation").
 *
 * For every active row b, with p = context_lens[b] (the position of the new token, 0-based):
 *   q_out[b,h,:]  = rope(q_in[b,h,:], p)   for all Hq heads   (q_out may alias q_in)
 *   k_cache[page, slot, h, :] = rope(k_new[b,h,:], p),  v_cache[page, slot, h, :] = v_new[b,h,:]
 *   for all Hkv heads, page = block_table[b, p / page_size], slot = p % page_size.
 * rope pairs element i with i + d/2 (i < d/2):  (x_i, x_{i+d/2}) -> (x_i c - x_{i+d/2} s,
 * x_{i+d/2} c + x_i s) with c = rope_cos[p, i], s = rope_sin[p, i].  Each result is the
 * round-to-nearest-even bf16 of the real value (products exact, one fp64 addition, one rounding), so
 * cache contents are reproducible bit for bit.  v is copied verbatim.
 *
 * Layout: q_in/q_out [B,Hq,d], k_new/v_new [B,Hkv,d] dense; cache element (page, slot, head, j) at
 * page*stride_page + slot*stride_token + head*stride_head + j (strides in elements);
 * block_table [B, max_pages_per_seq]; rope_cos/rope_sin [max_position, d/2].
 * A row whose position or page id is out of range writes nothing and sets status_flag bits (if
 * status_flag != NULL).  Two rows appending into the same slot is a caller error (not detected). */
int ac_rope_kv_append(const void* q_in, void* q_out, const void* k_new, const void* v_new,
                      void* k_cache, void* v_cache,
                      int64_t stride_page, int64_t stride_token, int64_t stride_head,
                      const int32_t* block_table, int max_pages_per_seq,
                      const int32_t* context_lens,
                      const float* rope_cos, const float* rope_sin, int max_position,
                      int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                      int32_t* status_flag, void* stream);

/* Prelude variants of A1 (the paper's attention-prelude family (i) names "optionally ... per-head
 * Q/K RMSNorm"; its per-model adaptations mention partial rotary embeddings).  Zero-initialise. */
typedef struct ac_rope_options {
    int rotary_dim;            /* 0 or d: rotate the whole vector; else even, < d: only elements
                                  [0, rotary_dim) are rotated, the rest pass through; the rope tables
                                  are then [max_position, rotary_dim/2] */
    int interleaved;           /* 0: pair element i with i + rotary_dim/2; 1: pair 2i with 2i + 1 */
    const void* q_norm_weight; /* device bf16 [d] or NULL: RMSNorm of every q head vector before the
                                  rotation: y = bf16(bf16(x / sqrt(mean(x^2) + eps)) * w) */
    const void* k_norm_weight; /* same for k (v is never normalised) */
    float norm_eps;
    int reserved[4];
} ac_rope_options;

/* ac_rope_kv_append with options (NULL = plain call).  Everything else as ac_rope_kv_append; the
 * rotation keeps its exact-then-round arithmetic, the norm is evaluated in fp64 (sum of squares,
 * square root and division correctly rounded) and rounded to bf16 where the formula above says. */
int ac_rope_kv_append_ex(const void* q_in, void* q_out, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache,
                         int64_t stride_page, int64_t stride_token, int64_t stride_head,
                         const int32_t* block_table, int max_pages_per_seq,
                         const int32_t* context_lens,
                         const float* rope_cos, const float* rope_sin, int max_position,
                         int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                         int32_t* status_flag, void* stream, const ac_rope_options* options);

/* Attention-prelude fusion, the paper's kernel family (i) ("QKV projection + RoPE"), with the KV
 * append of the kv_append kernel folded in: one launch computes
 *   y[b, n] = sum_k x[b, k] * w_qkv[n, k]     (bf16 operands, fp32 accumulation, rounded to bf16)
 * for n over the (Hq + 2 Hkv) * d output features (rows of w_qkv ordered q heads, k heads, v heads,
 * d rows per head; the [N, K] layout of the paper's decode GEMV), rotates the q and k features at
 * position context_lens[b] exactly as ac_rope_kv_append does, writes q to q_out [B,Hq,d] and k, v
 * into the cache slot block_table[b, p / page_size], p % page_size.  x is [B, H] bf16, H % 64 == 0.
 * The projection is not bit-reproducible against an fp64 evaluation (fp32 accumulation order): its
 * bf16 results can differ from the correctly rounded ones by one unit in the last place; the
 * rotation and the stores are exact given those results.  Errors and status bits as
 * ac_rope_kv_append.  Up to 16 batch rows run on a warp-level MMA kernel that streams w_qkv once
 * from HBM; larger batches run on a tcgen05 kernel (batch tiles of up to 128 rows as the M dimension
 * of the instruction, accumulators in tensor memory) that streams w_qkv once per 128 rows.  Both
 * give the same results up to fp32 accumulation order. */
int ac_qkv_rope_kv_append(const void* x, const void* w_qkv, int H, void* q_out,
                          void* k_cache, void* v_cache,
                          int64_t stride_page, int64_t stride_token, int64_t stride_head,
                          const int32_t* block_table, int max_pages_per_seq,
                          const int32_t* context_lens,
                          const float* rope_cos, const float* rope_sin, int max_position,
                          int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                          int32_t* status_flag, void* stream);

/* ac_qkv_rope_kv_append with the prelude variants of ac_rope_kv_append_ex (family (i) names the per-head
 * Q/K RMSNorm as an option of the fused prelude; the per-model adaptations mention partial rotary):
 * the projected, bf16-rounded q and k head vectors are normalised, rotated over their first
 * rotary_dim elements with the chosen pairing and stored, still in one launch.  The CTAs that share a
 * head (d/32 of the warp-MMA kernel, the one or two 32-pair tiles of the tcgen05 kernel) form a
 * thread-block cluster and exchange the sums of squares and the rotation partners through distributed
 * shared memory.  options == NULL (or all defaults) is ac_qkv_rope_kv_append.  The rope tables are
 * [max_position, rotary_dim/2].  Everything else as ac_qkv_rope_kv_append. */
int ac_qkv_rope_kv_append_ex(const void* x, const void* w_qkv, int H, void* q_out,
                             void* k_cache, void* v_cache,
                             int64_t stride_page, int64_t stride_token, int64_t stride_head,
                             const int32_t* block_table, int max_pages_per_seq,
                             const int32_t* context_lens,
                             const float* rope_cos, const float* rope_sin, int max_position,
                             int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                             int32_t* status_flag, void* stream, const ac_rope_options* options);

/* Output-projection fusion, the paper's kernel family (v) ("an output-projection (o_proj) kernel
 * fusing GEMV + residual + post-RMSNorm"), consuming the attention output:
 *   h[b, n]      = bf16( residual_in[b, n] + sum_k attn_out[b, k] * w_o[n, k] )   (fp32 sum, one rounding)
 *   normed[b, :] = RMSNorm(h[b, :]) * norm_weight = bf16( bf16( h / sqrt(mean(h^2) + eps) ) * w )
 * attn_out [B,K] bf16 (K = Hq*d, K % 64 == 0), w_o [N,K] bf16 ([N,K] layout, N % 32 == 0),
 * residual_in/residual_out/normed_out [B,N] bf16 (residual_out may alias residual_in), norm_weight
 * [N] bf16.  Two dependent launches on `stream`: the weight-streaming product with the residual add
 * in its epilogue, then the row norm (it needs all N features of a row); the second starts under the
 * first one's tail.  The norm is exact given h (fp64 sum of squares, correctly rounded sqrt and
 * division); h can differ from the correctly rounded value by one bf16 step (fp32 accumulation).
 * As for ac_qkv_rope_kv_append, B > 16 runs the product on the tcgen05 kernel. */
int ac_oproj_residual_rmsnorm(const void* attn_out, const void* w_o, int K, int N,
                              const void* residual_in, void* residual_out,
                              const void* norm_weight, float norm_eps, void* normed_out,
                              int B, void* stream);

/* A4: paged decode attention, family (iv).  Row b attends over tokens 0 .. n_b - 1 with
 * n_b = context_lens[b] + new_tokens (new_tokens = 1 right after ac_rope_kv_append, 0 to attend
 * over the cached tokens only); token t lives in page block_table[b, t / page_size], slot
 * t % page_size.  For query head hq:  out = softmax(scale * q_rot[b,hq,:] . K[t,:]) V  over those
 * tokens (bf16 operands, fp32 accumulation, fp32 softmax); softmax_scale <= 0 means 1/sqrt(d).
 *
 * Grid: one CTA per (request, KV head, split) holding the whole group of Hq/Hkv query heads.
 * num_splits == 1: the final bf16 result is written to out [B,Hq,d]; workspace may be NULL.
 * num_splits  > 1: out is not touched; split s writes its own normalised result to
 *   partial_o  = (float*)workspace                      [B,Hq,num_splits,d]
 *   partial_lse = partial_o + B*Hq*num_splits*d          [B,Hq,num_splits]  natural-log
 * log-sum-exp of the scaled scores; a split with no tokens writes lse = -inf and leaves its
 * partial_o untouched.  workspace_bytes must be >= ac_workspace_bytes(B,Hq,d,num_splits).
 * max_context_len must be >= every n_b (tokens beyond num_splits*split_tokens are not visited).
 * Contents of cache slots at or past n_b, of unreferenced pages and of unused block-table entries
 * never influence the result.  A page id outside [0, num_pages) reads as zeros. */
int ac_paged_decode_attn(const void* q_rot, const void* k_cache, const void* v_cache,
                         int64_t stride_page, int64_t stride_token, int64_t stride_head,
                         const int32_t* block_table, int max_pages_per_seq,
                         const int32_t* context_lens, int new_tokens, float softmax_scale,
                         int num_splits, void* workspace, size_t workspace_bytes, void* out,
                         int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                         int max_context_len, int32_t* status_flag, void* stream);

/* A4 + A5 in one launch: the same attention kernel, but the CTA that finishes last for a (request,
 * KV head) merges that pair's split partials itself and writes the final bf16 rows to out [B,Hq,d]
 * (the "fused cross-CTA merging" of family (iv); Supplementary Implementation Notes: "a fused
 * fence-based merge that removes a separate reduction kernel").  Each CTA publishes its partial,
 * fences, and takes a ticket from a per-(request, KV head) arrival counter; the holder of the last
 * ticket merges and resets the counter.  No CTA ever waits for another.  When a pair's splits number
 * at most 16 and the whole grid is resident at once, the launch instead makes each pair's splits one
 * thread-block cluster: every CTA stages its partial in its own shared memory and the CTA of split 0
 * reads them from there (distributed shared memory, two hardware cluster barriers; no partials in
 * global memory, no ticket); the workspace contract is the same either way.
 *
 * Arguments as ac_paged_decode_attn, except: out is always written; for num_splits > 1 the workspace
 * must hold ac_fused_workspace_bytes(B,Hq,Hkv,d,num_splits) bytes = the partials followed by int32
 * arrival counters [B,Hkv], and the counters must be ZERO on entry.  A launch that completes leaves
 * them zero, so call ac_fused_workspace_reset once after allocating the workspace (and again after
 * any launch that did not complete).  Results differ from the separate merge only in rounding order
 * of the fp32 combination; for fixed inputs and num_splits they are deterministic. */
size_t ac_fused_workspace_bytes(int B, int Hq, int Hkv, int d, int num_splits);
int ac_fused_workspace_reset(void* workspace, size_t workspace_bytes, int B, int Hq, int Hkv, int d,
                             int num_splits, void* stream);
int ac_paged_decode_attn_fused_merge(const void* q_rot, const void* k_cache, const void* v_cache,
                                     int64_t stride_page, int64_t stride_token, int64_t stride_head,
                                     const int32_t* block_table, int max_pages_per_seq,
                                     const int32_t* context_lens, int new_tokens, float softmax_scale,
                                     int num_splits, void* workspace, size_t workspace_bytes, void* out,
                                     int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                                     int max_context_len, int32_t* status_flag, void* stream);

/* A1 + A2 + A4 + A5 in ONE launch (the step as the paper's families (iii)/(iv) and its kv_append
 * kernel define it, fused): every CTA rotates the query rows of its group in registers (same exact
 * arithmetic as ac_rope_kv_append); the warp whose tile holds the new token's slot rotates k_new,
 * writes k and v into the cache page AND into the tile it just loaded, then attention proceeds over
 * context_lens[b] + 1 tokens and the last CTA of each (request, KV head) merges the splits.  Cache
 * contents after the call are bit-identical to ac_rope_kv_append's; outputs equal those of the
 * three-call sequence up to the fp32 merge order.
 *
 * q_in is the un-rotated query [B,Hq,d]; q_rot_out (optional, may be NULL) receives the rotated
 * rows and must not alias q_in.  Workspace as for ac_paged_decode_attn_fused_merge (counters zero on
 * entry when num_splits > 1).  A row whose position is outside the rope table or the block-table row,
 * whose page id is outside the pool, or whose context_lens[b] + 1 exceeds what the launch's split
 * grid covers (max_context_len too small for it: the new token's slot then lies in no CTA's range)
 * sets the status bits, appends nothing and writes no q_rot_out; its output is then unspecified. */
int ac_decode_step_fused(const void* q_in, void* q_rot_out, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache,
                         int64_t stride_page, int64_t stride_token, int64_t stride_head,
                         const int32_t* block_table, int max_pages_per_seq,
                         const int32_t* context_lens,
                         const float* rope_cos, const float* rope_sin, int max_position,
                         float softmax_scale, int num_splits, void* workspace, size_t workspace_bytes,
                         void* out, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                         int max_context_len, int32_t* status_flag, void* stream);

/* Options of the _ex entry points.  Zero-initialise; unknown fields must stay zero. */
typedef struct ac_attn_options {
    int window;      /* > 0: sliding-window attention -- row b attends over its last `window` tokens
                        only, i.e. tokens max(0, n_b - window) .. n_b - 1 (the paper wires a sliding
                        window in for one of its model families, "Per-Model Adaptations"); 0: all */
    int fused_merge; /* ac_paged_decode_attn_ex only: non-zero = behave as ac_paged_decode_attn_fused_merge */
    const int32_t* row_order; /* optional device array [B], a permutation of 0..B-1: grid row y serves
                        request row_order[y].  CTAs are dispatched in grid order, so listing the requests
                        by decreasing context length (what a scheduler that knows the lengths can do
                        for free) shortens the tail of grids that are several waves deep.  Any
                        permutation gives the same results.  NULL: the kernel ranks the requests
                        itself when B <= 128 and serves them in index order otherwise. */
    const struct ac_rope_options* rope; /* ac_decode_step_fused_ex only: prelude variants (per-head Q/K
                        RMSNorm, partial rotary, interleaved pairing) applied to q_in and k_new inside the
                        step, with the arithmetic and the table shapes of ac_rope_kv_append_ex; NULL or
                        all-default options = the plain rotation */
    int reserved[2];
} ac_attn_options;

/* ac_paged_decode_attn / ac_paged_decode_attn_fused_merge / ac_decode_step_fused with options
 * (options == NULL means defaults).  With a window, tokens before the window's start are neither
 * read (whole tiles) nor weighted (the first tile masks them), so their pages may already have been
 * recycled; the splits partition the at most window + 63 tokens from the window's start rounded
 * down to a multiple of 64, so pass min(max_context_len, window + 63) to ac_decode_plan. */
int ac_paged_decode_attn_ex(const void* q_rot, const void* k_cache, const void* v_cache,
                            int64_t stride_page, int64_t stride_token, int64_t stride_head,
                            const int32_t* block_table, int max_pages_per_seq,
                            const int32_t* context_lens, int new_tokens, float softmax_scale,
                            int num_splits, void* workspace, size_t workspace_bytes, void* out,
                            int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                            int max_context_len, int32_t* status_flag, void* stream,
                            const ac_attn_options* options);
int ac_decode_step_fused_ex(const void* q_in, void* q_rot_out, const void* k_new, const void* v_new,
                            void* k_cache, void* v_cache,
                            int64_t stride_page, int64_t stride_token, int64_t stride_head,
                            const int32_t* block_table, int max_pages_per_seq,
                            const int32_t* context_lens,
                            const float* rope_cos, const float* rope_sin, int max_position,
                            float softmax_scale, int num_splits, void* workspace, size_t workspace_bytes,
                            void* out, int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                            int max_context_len, int32_t* status_flag, void* stream,
                            const ac_attn_options* options);

/* A5: merge of the split partials ("cross-CTA merging" of family (iv), here as its own kernel):
 *   M = max_s lse_s,  w_s = exp(lse_s - M),  out[b,hq,:] = sum_s w_s partial_o[b,hq,s,:] / sum_s w_s
 * rounded to bf16.  Splits with lse = -inf are skipped (their partial_o is not read); a row whose
 * splits are all empty, or with context_lens[b] < 0 (context_lens may be NULL), gets +0.
 * workspace has the layout written by ac_paged_decode_attn for the same B, Hq, d, num_splits. */
int ac_splitkv_merge(const void* workspace, int num_splits, const int32_t* context_lens, void* out,
                     int B, int Hq, int d, void* stream);

/* The whole step from HOST buffers (for callers that hold the step's inputs on the host, and for
 * end-to-end timing): copies q/k_new/v_new/block_table/context_lens from the *_host buffers (pinned
 * memory recommended) into the caller's device buffers of the same name, resets the arrival
 * counters, enqueues ac_decode_step_fused for the given num_splits (workspace_bytes >=
 * ac_fused_workspace_bytes), and delivers the bf16 result in out AND out_host (when out_host is pinned
 * memory the GPU can address, the kernel's final stores go to both; otherwise a copy from out follows).  When the host
 * buffers are pinned memory the GPU can address and their sizes are multiples of 16 bytes, the five
 * inputs are gathered (and the counters cleared) by ONE small kernel reading host memory directly
 * instead of five copy-engine transfers; otherwise each buffer gets its own cudaMemcpyAsync.  The
 * *_host inputs must be complete when the call is made and stay unchanged until the step has
 * finished: that kernel reads them as soon as it is resident, which may be while earlier work of the
 * stream is still running (it writes the device buffers only after that work has completed).
 * Everything is asynchronous on `stream`; the caller
 * synchronises the stream before reading out_host.  The KV cache pools and rope tables stay on the
 * device (they are the layer's resident state, not a per-step input).  No paper counterpart. */
int ac_decode_step_host(const void* q_host, const void* k_new_host, const void* v_new_host,
                        const int32_t* block_table_host, const int32_t* context_lens_host,
                        void* out_host,
                        void* q, void* k_new, void* v_new, int32_t* block_table,
                        int32_t* context_lens, void* out,
                        void* k_cache, void* v_cache,
                        int64_t stride_page, int64_t stride_token, int64_t stride_head,
                        int max_pages_per_seq,
                        const float* rope_cos, const float* rope_sin, int max_position,
                        float softmax_scale, int num_splits, void* workspace, size_t workspace_bytes,
                        int B, int Hq, int Hkv, int d, int page_size, int num_pages,
                        int max_context_len, int32_t* status_flag, void* stream);

/* Calibration helper (no paper counterpart): enqueues a plain coalesced read-only pass over
 * buffer[0, bytes) -- 16-byte streaming loads, nothing written -- on `stream`.  Timed by the caller
 * (CUDA events around it) it gives the read-only HBM ceiling of the machine, which a benchmark can
 * print beside the copy-measured peak its roofline fractions use.  buffer: device memory, 16-byte
 * aligned, bytes >= 16 (a tail shorter than 16 bytes is not read); sink: optional device word that
 * receives the fold of a thread's loads only if that happens to equal one constant (it keeps the
 * loads alive; expect it untouched).  ac_init must have succeeded on the current device. */
int ac_hbm_read_probe(const void* buffer, size_t bytes, void* sink, void* stream);

/* Size of the library's built-in partial-result array (bytes), held by every GPU that loads the
 * library until the process exits. */
#define AC_STATIC_SCRATCH_BYTES (8u << 20)

/* Split-KV attention and merge in one call, for callers that cannot allocate device memory.  (The
 * paper has no counterpart to this entry point; it exists for the integration cases below.)
 *
 * ac_paged_decode_attn needs a workspace for the split partials, which normally means a cudaMalloc
 * (or a framework allocation) somewhere in the caller.  That is not always possible: an engine that
 * gave all remaining HBM to its KV-cache pool at start-up has nothing left to ask for; code running
 * under a host framework that forbids allocation in the serving loop, or that must not take the
 * driver's allocation lock, cannot call cudaMalloc at all; and a stateless step function has nowhere
 * to keep a buffer from one call to the next.  This entry point calls no cudaMalloc, cudaFree or
 * any allocating routine: the partials go into a fixed array inside the library image, of
 * AC_STATIC_SCRATCH_BYTES bytes per GPU.
 *
 * Arguments are those of ac_paged_decode_attn without workspace/workspace_bytes; the caller still
 * passes every input and the output.  The call runs the attention kernel with num_splits splits
 * (use ac_decode_plan to choose) and then the merge, both on `stream`, and always writes the final
 * bf16 rows to out [B,Hq,d].
 *
 * Limits and rules
 *   - For num_splits > 1, B * Hq * num_splits * (d + 1) * 4 bytes must not exceed
 *     AC_STATIC_SCRATCH_BYTES, otherwise AC_ERR_SCRATCH_LIMIT is returned and nothing is launched.
 *     Lower num_splits, or use ac_paged_decode_attn with your own workspace.  A single split uses
 *     no scratch (the attention kernel writes `out` itself), so no size limit applies to it.
 *   - ac_init must have succeeded on the current device.  The first call on each device also looks
 *     up the array's device address (once; later calls reuse it): make that first call outside any
 *     stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call wrote.
 *     Nothing needs clearing between calls (each call overwrites the log-sum-exp slot of every split
 *     it uses before reading it, and never reads the partial of a split marked empty), but two calls
 *     whose kernels overlap on the GPU -- different streams, or different host threads without
 *     ordering between their streams -- would write the same bytes and corrupt each other.  Order
 *     them on one stream or with events.
 *   - Errors are otherwise those of ac_paged_decode_attn and ac_splitkv_merge. */
int ac_paged_decode_attn_static_scratch(const void* q_rot, const void* k_cache, const void* v_cache,
                                        int64_t stride_page, int64_t stride_token, int64_t stride_head,
                                        const int32_t* block_table, int max_pages_per_seq,
                                        const int32_t* context_lens, int new_tokens,
                                        float softmax_scale, int num_splits, void* out, int B, int Hq,
                                        int Hkv, int d, int page_size, int num_pages,
                                        int max_context_len, int32_t* status_flag, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AC_H_ */

/*
 * opt_gqa.h -- C ABI of the Opt-GQA attention library for NVIDIA B200 (sm_100a).
 *
 * Grouped-query attention in which the G = Hq / Hkv query heads of a group share
 * one K/V head, K/V live in a paged (block-table) cache, and an ALiBi linear bias
 * is added to the scores:
 *
 *     out[t,h,:] = sum_j softmax_j( scale * <q[t,h], k_j> - slope_h * (pos_t - j) ) * v_j
 *
 * with k_j, v_j the j-th cached token of the sequence, head h / G.
 *
 * Conventions common to every call
 *  - Every pointer is a DEVICE pointer owned by the caller unless the argument is
 *    documented as HOST.  The library allocates nothing and keeps no pointer after
 *    the call returns; calls only enqueue work on `stream` (a cudaStream_t passed as
 *    void*, NULL = the default stream) and return.  The caller keeps every buffer
 *    alive until that work has finished.  `stream` must belong to the current device.
 *  - State of the library, all of it per device: one status word in device memory
 *    (opt_gqa_device_status), the fixed scratch array of the _no_alloc entry point, and
 *    host-side caches of symbol addresses and kernel attributes filled by the first call
 *    on a device (make that call outside stream capture).  The caches are atomics: calls
 *    from several host threads are safe, also when they are the first ones.
 *  - Ordering inside a stream: the kernels are launched with programmatic stream
 *    serialisation and wait for the preceding kernel of the stream before they read
 *    anything it may write (q, k_new, v_new, the cache, the partials) or overwrite
 *    anything it may read (out, the workspace).  Two index arrays are the exception:
 *    block_tables and context_lens are read BEFORE that wait (the split of the work is
 *    computed from them while the preceding kernel drains).  They must therefore not be
 *    produced by a kernel that signals its dependents early (griddepcontrol
 *    .launch_dependents / cudaTriggerProgrammaticLaunchCompletion); no kernel of this
 *    library writes them except the gather of opt_gqa_decode_step_host, which does not
 *    signal early.  Ordinary producers (copies, kernels without that signal) are fine.
 *  - dtype: OPT_GQA_FP32 (0) or OPT_GQA_BF16 (1).  q, k_new/v_new, the cache and out
 *    share it.  Slopes, scale, partials are always fp32.  All arithmetic is fp32;
 *    results are rounded once (to nearest even) when stored.
 *  - Cache layout: k_cache, v_cache are [num_blocks, Hkv, bs, D] row-major: one
 *    (page, kv head) is one contiguous chunk of bs*D elements.
 *  - Supported shapes: D in {64, 128}; bs in {16, 32}; G = Hq/Hkv in {1, 2, 4, 8}.
 *  - Data pointers must be 16-byte aligned.
 *  - Return value: 0 (OPT_GQA_OK) or a negative OPT_GQA_ERR_* code.  Argument checks
 *    are done on the host before anything is enqueued; a failed check enqueues
 *    nothing.  B = 0 or T = 0 returns OK without a launch.  There are no device
 *    traps: a device-side wait that runs out records OPT_GQA_ERR_TIMEOUT in a status
 *    word read by opt_gqa_device_status().
 *  - Contract on index data (not checked on the device): context_lens[s] >= 0;
 *    block_tables[s][i] is a valid page id for i < ceil(context_lens[s] / bs), and is
 *    never read beyond that; slot_mapping entries are < num_blocks*bs and distinct
 *    within one call (negative = skip the token).
 *  - The tail of a sequence's last page and pages no sequence uses are never
 *    interpreted: results do not depend on their contents (NaN bit patterns included).
 */
#ifndef OPT_GQA_H_
#define OPT_GQA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OPT_GQA_FP32 0
#define OPT_GQA_BF16 1

#define OPT_GQA_OK 0
#define OPT_GQA_ERR_NULL (-1)    /* a required pointer is NULL                            */
#define OPT_GQA_ERR_SHAPE (-2)   /* unsupported or inconsistent sizes                     */
#define OPT_GQA_ERR_DTYPE (-3)   /* dtype is neither OPT_GQA_FP32 nor OPT_GQA_BF16        */
#define OPT_GQA_ERR_ALIGN (-4)   /* a data pointer is not 16-byte aligned                 */
#define OPT_GQA_ERR_CUDA (-5)    /* the CUDA runtime refused the launch or a copy         */
#define OPT_GQA_ERR_TIMEOUT (-6) /* a bounded device-side wait ran out (device status)    */
#define OPT_GQA_ERR_SCRATCH (-7) /* the call needs more than OPT_GQA_STATIC_SCRATCH_BYTES  */

/* Size of the scratch array built into the library for opt_gqa_paged_attention_decode_no_alloc. */
#define OPT_GQA_STATIC_SCRATCH_BYTES (8u << 20)

/*
 * Slot-mapped write of new tokens' K/V into the paged cache: Algorithm 1,
 * "Reshape and store K, V into C_K, C_V" (same step in Algorithm 2; Eq. 2: the
 * cached sequence is the earlier tokens followed by the new ones).
 *
 *   k_new, v_new  [T, Hkv, D]        rows of the T new tokens
 *   k_cache, v_cache                 the pool, modified in place
 *   slot_mapping  [T] int64          slot = page*bs + offset; token t goes to
 *                                    cache[slot/bs][h][slot%bs][:] for every h;
 *                                    a negative slot skips the token
 * A bit-exact copy.  Call it before the attention call of the same step, on the
 * same stream: context_lens passed to attention already counts these tokens.
 */
int opt_gqa_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                         const int64_t* slot_mapping, int T, int Hkv, int D, int bs,
                         int64_t num_blocks, int dtype, void* stream);

/*
 * Decode attention over the paged cache, one query token per sequence at position
 * n_s - 1: Algorithm 2, "Compute context attention with caches"; scores by Eq. 3
 * (scaled dot product plus the ALiBi bias -slope_h*(n_s-1-j) of the "Integration
 * and Optimization of ALiBi" paragraph), softmax by Eq. 4, weighted sum of V by
 * Eq. 5; heads grouped as in "Query Grouping" / "Shared Key-Value" (query head h
 * reads K/V head h / G).
 *
 *   out           [B, Hq, D]         written when partition_size == 0
 *   q             [B, Hq, D]
 *   block_tables  [B, max_blocks_per_seq] int32
 *   context_lens  [B] int32          n_s, counts the current token; n_s == 0 gives
 *                                    zero rows
 *   alibi_slopes  [Hq] fp32, or NULL for no bias
 *   partition_size  0: one CTA walks the whole sequence and writes out.
 *                   P > 0 (a multiple of 16): the long-sequence split described
 *                   before Eq. 1 -- work item (s, kv head, p) attends to keys
 *                   [pP, min((p+1)P, n_s)) and writes, for each head of the group,
 *                   the normalised partial result and its log-sum-exp:
 *                     partial_out [B, Hq, max_partitions, D] fp32
 *                     partial_lse [B, Hq, max_partitions]    fp32 (natural log)
 *                   for p < ceil(n_s / P); other entries are left untouched.  out
 *                   is not written; follow with opt_gqa_paged_attention_reduce.
 *                   max_partitions >= ceil(max_s n_s / P) is the caller's promise.
 */
int opt_gqa_paged_attention_decode(void* out, const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* block_tables, int max_blocks_per_seq,
                                   const int32_t* context_lens, const float* alibi_slopes, float scale,
                                   int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                                   int partition_size, float* partial_out, float* partial_lse,
                                   int max_partitions, int dtype, void* stream);

/*
 * The same operation, arguments and results as opt_gqa_paged_attention_decode, forced
 * onto the CUDA-core kernel (16 lanes per token row, warp-shuffle reduce-scatter of the
 * G partial dot products, packed fp32 FMAs).  opt_gqa_paged_attention_decode uses this
 * kernel for fp32 caches and a tensor-core tile kernel (the query group as the rows of
 * m16n8k16 tiles) for bf16 caches; this entry point keeps the CUDA-core form of Eq. 3-5
 * reachable for bf16 as well, for comparison and as a cross-check.
 */
int opt_gqa_paged_attention_decode_simt(void* out, const void* q, const void* k_cache, const void* v_cache,
                                        const int32_t* block_tables, int max_blocks_per_seq,
                                        const int32_t* context_lens, const float* alibi_slopes, float scale,
                                        int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                                        int partition_size, float* partial_out, float* partial_lse,
                                        int max_partitions, int dtype, void* stream);

/*
 * Partitioned decode with a load-balanced split, bf16 caches only: the same result as
 * opt_gqa_paged_attention_decode with partition_size = P followed by the reduce, but the
 * context partitions (the split described before Eq. 1) are additionally cut wherever the
 * share of one worker of the persistent grid ends, so that every SM streams the same number
 * of cache bytes whatever the mix of sequence lengths.  Every piece lies inside one
 * P-token partition of one (sequence, KV head); its normalised result and log-sum-exp go
 * to `workspace` in a layout private to the library, and
 * opt_gqa_paged_attention_reduce_balanced (same B, Hq, Hkv, D, partition_size,
 * max_partitions, same workspace, later on the same stream) merges them into out.
 *
 *   workspace     device memory, 16-byte aligned; contents need no initialisation and are overwritten
 *   workspace_bytes  HOST value: the size of `workspace`; OPT_GQA_ERR_SHAPE if it is below what the
 *                 split of these sizes needs (opt_gqa_workspace_bytes(B, Hq, D, max_partitions) always
 *                 suffices)
 *   partition_size  P > 0, a multiple of 16;  max_partitions >= ceil(max_s n_s / P)
 * Other arguments as in opt_gqa_paged_attention_decode.  dtype must be OPT_GQA_BF16.
 */
int opt_gqa_paged_attention_decode_balanced(const void* q, const void* k_cache, const void* v_cache,
                                            const int32_t* block_tables, int max_blocks_per_seq,
                                            const int32_t* context_lens, const float* alibi_slopes, float scale,
                                            int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                                            int partition_size, void* workspace, size_t workspace_bytes,
                                            int max_partitions, int dtype, void* stream);

/*
 * Log-sum-exp merge of the pieces written by opt_gqa_paged_attention_decode_balanced (the
 * combination step of the paragraph before Eq. 1, over pieces instead of whole partitions):
 *     out = sum_c e^{lse_c} o_c / sum_c e^{lse_c}   over the pieces c of the row's sequence and KV head.
 * out [B, Hq, D] in `dtype`; n_s == 0 gives zero rows.
 */
int opt_gqa_paged_attention_reduce_balanced(void* out, const void* workspace, size_t workspace_bytes,
                                            const int32_t* context_lens, int B, int Hq, int Hkv, int D,
                                            int partition_size, int max_partitions, int dtype, void* stream);

/*
 * Merge of the partitions' results (the paragraph before Eq. 1: each partition's
 * output is kept and then combined into the result for the whole sequence):
 *     out = sum_p e^{lse_p} o_p / sum_p e^{lse_p},   p < ceil(n_s / P)
 * evaluated with the largest lse subtracted.  n_s == 0 gives zero rows.
 * Arguments as written by opt_gqa_paged_attention_decode with the same
 * partition_size and max_partitions.
 */
int opt_gqa_paged_attention_reduce(void* out, const float* partial_out, const float* partial_lse,
                                   const int32_t* context_lens, int B, int Hq, int D, int partition_size,
                                   int max_partitions, int dtype, void* stream);

/*
 * Partitioned decode and merge in one call, for callers that cannot provide a
 * workspace.  (The paper has no counterpart: this is a packaging variant of the two
 * calls above.)  Some hosts of the library cannot allocate device memory where they
 * call it -- code running inside an engine that has already given all free memory to
 * the cache pool, or in a callback where cudaMalloc is off limits because it
 * synchronises the device.  This entry point allocates nothing, neither on the host nor
 * on the device: the partitions' partial results go to a fixed array of
 * OPT_GQA_STATIC_SCRATCH_BYTES (8 MiB) that is part of the loaded library.
 *
 * Result: the same out [B, Hq, D] as opt_gqa_paged_attention_decode with partition_size
 * = P > 0 followed by opt_gqa_paged_attention_reduce; arguments as there.
 *
 *  - Limit: B * Hq * max_partitions * (D + 1) * 4 bytes must fit in the array;
 *    otherwise OPT_GQA_ERR_SCRATCH is returned and nothing is enqueued.
 *  - The array exists once per GPU, from the first use of the library on that GPU until
 *    the process exits, and all calls on that GPU share it: calls that can overlap on the
 *    GPU (different streams, no ordering between them) race on it.  It needs no clearing;
 *    what a previous call left in it is never read.
 *  - The first call on each device looks up the array's device address (a runtime call
 *    made with that device current); make that first call outside any stream capture.
 *    The address belongs to the CURRENT device: `stream` must be a stream of that device.
 */
int opt_gqa_paged_attention_decode_no_alloc(void* out, const void* q, const void* k_cache, const void* v_cache,
                                            const int32_t* block_tables, int max_blocks_per_seq,
                                            const int32_t* context_lens, const float* alibi_slopes, float scale,
                                            int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                                            int partition_size, int max_partitions, int dtype, void* stream);

/*
 * Multi-token (chunked-prefill) variant on tensor cores: the prompt branch of
 * Algorithms 1 and 2 run over the paged cache with a causal mask plus the ALiBi
 * bias ("Create ALiBi bias"; Eq. 3-5).  Sequence s contributes
 * q_len_s = q_start_loc[s+1] - q_start_loc[s] new tokens whose K/V are already in
 * the cache; new token i sits at position pos = n_s - q_len_s + i and attends to
 * keys j <= pos with bias -slope_h*(pos - j).
 *
 *   out, q        [total_q_tokens, Hq, D]  (bf16 only)
 *   q_start_loc   [B+1] int32              prefix sums of q_len_s, device memory
 *   total_q_tokens HOST value: rows of q and out (= q_start_loc[B]); rows are read up to it
 *   max_q_len     HOST value >= max_s q_len_s (sizes the grid)
 * Runs on tcgen05.mma with accumulators in tensor memory, for both head dimensions and any scale (a
 * negative scale negates Q inside the instruction, a zero scale leaves the dot products out).
 */
int opt_gqa_paged_attention_prefill(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                                    int max_q_len, const void* k_cache, const void* v_cache,
                                    const int32_t* block_tables, int max_blocks_per_seq, const int32_t* context_lens,
                                    const float* alibi_slopes, float scale, int B, int Hq, int Hkv, int D, int bs,
                                    int64_t num_blocks, int dtype, void* stream);

/*
 * The same operation, arguments and results as opt_gqa_paged_attention_prefill, forced onto the
 * warp-level kernel (mma.sync m16n8k16, eight consumer warps of 16 rows each and a producer warp):
 * keeps the earlier form of Eq. 3-5 reachable as a cross-check and for comparison.
 */
int opt_gqa_paged_attention_prefill_mma(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                                        int max_q_len, const void* k_cache, const void* v_cache,
                                        const int32_t* block_tables, int max_blocks_per_seq,
                                        const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                        int Hq, int Hkv, int D, int bs, int64_t num_blocks, int dtype, void* stream);

/*
 * Decode and chunked prefill with a local (sliding-window) mask: Algorithm 1, "Create causal and
 * local attention masks" -- the branch taken when no ALiBi slopes are given, although slopes are
 * accepted here as well.  The token at position pos attends to keys pos - window < j <= pos only;
 * everything else is as in Eq. 3-5.  Neither mask exists in memory: the window moves the first tile
 * a sequence's stream (or a query block's key range) starts at, and the edge tile is masked from the
 * indices.
 *
 * opt_gqa_paged_attention_decode_local: split decode and merge in one call, out [B, Hq, D] is written,
 * partition_size > 0.  bf16 caches take the balanced split (arguments as
 * opt_gqa_paged_attention_decode_balanced followed by opt_gqa_paged_attention_reduce_balanced); fp32 caches
 * one partial per partition on the CUDA-core kernel, partial_out [B, Hq, max_partitions, D] followed by
 * partial_lse at the start of the workspace (workspace_bytes >= B * Hq * max_partitions * (D + 1) * 4),
 * and the merge skips the partitions that lie wholly before the window.
 * opt_gqa_paged_attention_prefill_local: arguments as opt_gqa_paged_attention_prefill (bf16).
 * window > 0 is required.
 */
int opt_gqa_paged_attention_decode_local(void* out, const void* q, const void* k_cache, const void* v_cache,
                                         const int32_t* block_tables, int max_blocks_per_seq,
                                         const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                         int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                                         void* workspace, size_t workspace_bytes, int max_partitions, int window,
                                         int dtype, void* stream);

int opt_gqa_paged_attention_prefill_local(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                                          int max_q_len, const void* k_cache, const void* v_cache,
                                          const int32_t* block_tables, int max_blocks_per_seq,
                                          const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                          int Hq, int Hkv, int D, int bs, int64_t num_blocks, int window, int dtype,
                                          void* stream);

/*
 * The prompt branch with empty caches (Algorithms 1 and 2: "Caches are empty" -> "Adjust Q, K, V
 * for GQA grouping", "Create ALiBi bias", then Eq. 3-5): every sequence attends causally to its own
 * new tokens, read from contiguous tensors instead of the paged cache.  Token i of sequence s
 * (row q_start_loc[s] + i) sees keys 0 .. i of that sequence with bias -slope_h*(i - j); query
 * head h uses K/V head h / G.  The same tcgen05 kernel as opt_gqa_paged_attention_prefill (D 64 or 128,
 * any scale), with K/V tiles fetched through 3-D tensor maps over k and v.  (Writing k, v into the cache for later
 * decode steps is opt_gqa_cache_append, before or after this call.)
 *
 *   out, q        [total_q_tokens, Hq, D]   bf16
 *   k, v          [total_q_tokens, Hkv, D]  bf16
 *   q_start_loc   [B+1] int32               prefix sums of the sequences' lengths, device memory
 *   total_q_tokens, max_q_len               HOST values, as in opt_gqa_paged_attention_prefill
 *   alibi_slopes  [Hq] fp32 or NULL (causal mask only)
 */
int opt_gqa_prompt_attention(void* out, const void* q, const void* k, const void* v, const int32_t* q_start_loc,
                             int total_q_tokens, int max_q_len, const float* alibi_slopes, float scale, int B, int Hq,
                             int Hkv, int D, int dtype, void* stream);

/*
 * Q/K/V projection of Eq. 1 (Q = X W_Q, K = X W_K, V = X W_V) for the T tokens of a decode step, from
 * 4-bit group-quantised weights, with the keys and values written where the rest of the step reads them:
 * Algorithm 1, "Reshape and store K, V into C_K, C_V".  The paper names GPTQ in its title and gives no
 * storage format; the interchange layout taken here is the common group-wise one, W [K, N] with the
 * three matrices side by side (columns 0 .. Hq D - 1 query, then Hkv D key, then Hkv D value):
 *
 *   qweight  [K/8, N]    uint32   code of row 8r+i, column n in bits 4i .. 4i+3 of word (r, n)
 *   scales   [K/gs, N]   bf16
 *   qzeros   [K/gs, N/8] uint32   zero point of group g, column 8c+i in bits 4i .. 4i+3 of word (g, c)
 *   w[k][n] = scales[k/gs][n] * (code[k][n] - zero[k/gs][n]),   y[t][n] = sum_k x[t][k] w[k][n]
 *
 * opt_gqa_int4_prepack rewrites these three arrays once into the layout the kernel streams (`packed`,
 * opt_gqa_int4_packed_bytes(K, N, gs) bytes of device memory, 16-byte aligned; all four DEVICE pointers).
 * K a multiple of gs, gs 64 or 128, N a multiple of 32.  opt_gqa_int4_packed_bytes returns 0 otherwise.
 *
 * opt_gqa_qkv_project_int4: x [T, K] bf16 (K = the model width), N = (Hq + 2 Hkv) D.
 *   q_out          [T, Hq, D]  bf16, always written
 *   k_out, v_out   [T, Hkv, D] bf16, or both NULL
 *   k_cache, v_cache           the paged pool [num_blocks, Hkv, bs, D] bf16, or both NULL; token t's key and
 *                              value go to slot_mapping[t] exactly as in opt_gqa_cache_append (a negative
 *                              slot, or one past the pool, skips the token)
 * At least one of the two destinations for K/V must be given.  Sums are accumulated in fp32 and rounded
 * once to bf16.  The kernel is sized for the few tokens of a decode step (up to 16 per pass over the
 * weights); larger T is accepted and takes one pass per 16 tokens.  All pointers are DEVICE pointers,
 * 16-byte aligned.  Errors as everywhere in this header; nothing is launched on an error.
 */
size_t opt_gqa_int4_packed_bytes(int K, int N, int gs);

int opt_gqa_int4_prepack(void* packed, const uint32_t* qweight, const void* scales, const uint32_t* qzeros, int K,
                         int N, int gs, void* stream);

int opt_gqa_qkv_project_int4(void* q_out, void* k_out, void* v_out, void* k_cache, void* v_cache,
                             const int64_t* slot_mapping, const void* x, const void* packed, int T, int K, int Hq,
                             int Hkv, int D, int bs, int64_t num_blocks, int gs, void* stream);

/*
 * One decode step of the attention layer, Algorithm 2 from "Store reshaped K, V
 * into C_K, C_V" to "Compute context attention with caches": cache_append of the
 * B new tokens (k_new, v_new [B, Hkv, D], slot_mapping [B]), then decode, then --
 * when partition_size > 0 -- the reduce, all enqueued on `stream` by one call.
 * workspace: workspace_bytes (a HOST value) bytes of device memory, 16-byte aligned;
 * opt_gqa_workspace_bytes(B, Hq, D, max_partitions) suffices, less than the step needs
 * is refused with OPT_GQA_ERR_SHAPE before anything is enqueued; may be NULL (and 0)
 * when partition_size is 0.  bf16 caches take
 * the balanced split (decode_balanced + reduce_balanced), fp32 caches one partial
 * per partition (partial_out followed by partial_lse at the start of workspace).
 * Other arguments as in the calls it chains.  out [B, Hq, D] is always written.
 * A bf16 step whose contexts are all short (max_partitions * partition_size <= 2048) and whose (sequence, KV
 * head) streams number between 1.5 and 4 times the GPU's multiprocessors runs as a single launch: one CTA per
 * stream walks the whole context, stores the stream's new token itself and writes out (the result is the same;
 * the workspace is not touched).
 * On the bf16 split path with at most 1024 (sequence, KV head) streams no separate append kernel
 * runs: the decode kernel stores sequence s's new token to slot_mapping[s] itself, just before it
 * fetches the tile that holds position context_lens[s] - 1 (a sequence with context_lens 0 has no
 * such tile and stores nothing).
 */
int opt_gqa_decode_step(void* out, const void* q, const void* k_new, const void* v_new,
                        const int64_t* slot_mapping, void* k_cache, void* v_cache, const int32_t* block_tables,
                        int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes,
                        float scale, int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                        int partition_size, void* workspace, size_t workspace_bytes, int max_partitions, int dtype,
                        void* stream);

/*
 * The same step for a caller whose per-step tensors live in HOST memory (pinned,
 * for the copies to be asynchronous): out_host, q_host, k_new_host, v_new_host,
 * slot_mapping_host, block_tables_host, context_lens_host are HOST pointers with
 * the shapes above.  They are copied to `staging` (device memory of
 * opt_gqa_step_staging_bytes(...) bytes, 256-byte aligned) on `stream`, the step
 * runs there, and out is copied back to out_host; the call returns once everything
 * is enqueued, so synchronise `stream` before reading out_host or reusing the host
 * buffers.  The cache, alibi_slopes and workspace stay DEVICE pointers: the cache
 * is state that persists between steps.  Page-locked (pinned, mapped) host buffers are
 * read by one gather kernel and out is stored into out_host by the step's last kernel;
 * pageable buffers are moved with cudaMemcpyAsync instead.  (Convenience wrapper around the
 * step; the transfers are the "Reshape Q, K, V" hand-over of Algorithm 2's inputs.)
 */
int opt_gqa_decode_step_host(void* out_host, const void* q_host, const void* k_new_host, const void* v_new_host,
                             const int64_t* slot_mapping_host, const int32_t* block_tables_host,
                             const int32_t* context_lens_host, void* staging, void* k_cache, void* v_cache,
                             int max_blocks_per_seq, const float* alibi_slopes, float scale, int B, int Hq,
                             int Hkv, int D, int bs, int64_t num_blocks, int partition_size, void* workspace,
                             size_t workspace_bytes, int max_partitions, int dtype, void* stream);

/*
 * opt_gqa_decode_step_host for a caller that has looked the device-side addresses of its page-locked
 * buffers up once (cudaHostGetDevicePointer; with unified addressing, memory from cudaHostAlloc /
 * cudaMallocHost has the same address on both sides): the seven *_view arguments are those addresses,
 * the call makes no pointer queries, and the transfers are always done by the kernels themselves (one
 * gather kernel in, out stored by the step's last kernel).  Views must be 4-byte aligned, out_view
 * 16-byte aligned (OPT_GQA_ERR_ALIGN otherwise).  Everything else as in opt_gqa_decode_step_host.
 */
int opt_gqa_decode_step_mapped(void* out_view, const void* q_view, const void* k_new_view, const void* v_new_view,
                               const int64_t* slot_mapping_view, const int32_t* block_tables_view,
                               const int32_t* context_lens_view, void* staging, void* k_cache, void* v_cache,
                               int max_blocks_per_seq, const float* alibi_slopes, float scale, int B, int Hq,
                               int Hkv, int D, int bs, int64_t num_blocks, int partition_size, void* workspace,
                               size_t workspace_bytes, int max_partitions, int dtype, void* stream);

/* Device bytes opt_gqa_decode_step_host needs in `staging`.  Host arithmetic; 0 for bad arguments. */
size_t opt_gqa_step_staging_bytes(int B, int Hq, int Hkv, int D, int max_blocks_per_seq, int dtype);

/*
 * Bytes of device scratch a split decode needs, whichever layout is used: one
 * (D+1)-float row per (sequence, head, partition) -- partial_out followed by
 * partial_lse -- or the balanced split's piece rows and bookkeeping, which add a
 * fixed 16384 rows and less than 1 KB + 16*B bytes.  (Workspace sizing for the
 * partitioning step; pure host arithmetic.)  Returns 0 for non-positive arguments.
 */
size_t opt_gqa_workspace_bytes(int B, int Hq, int D, int max_partitions);

/*
 * Diagnostics for the bounded waits (no counterpart in the paper).  Every wait of a kernel on an
 * mbarrier gives up after about 2^28 SM clocks, records OPT_GQA_ERR_TIMEOUT in the status word and
 * lets the kernel return.  This call makes exactly that happen, so that a host's handling of the
 * status can be tested without a fault or a hang: it launches one warp on `stream` that waits, with
 * a limit of limit_cycles SM clocks (1 .. 2^24; OPT_GQA_ERR_SHAPE otherwise), for bytes that nothing
 * sends.  After the stream has drained opt_gqa_device_status() returns OPT_GQA_ERR_TIMEOUT once.
 */
int opt_gqa_debug_wait_timeout(long long limit_cycles, void* stream);

/*
 * Read-only streaming probe (diagnostics; no counterpart in the paper): streams `bytes` bytes from
 * src through the same per-warp rings of bulk async copies, in the same grid shape, as the decode
 * kernels, with no arithmetic attached -- the rate it reaches is the ceiling of that data path on
 * this GPU.  bytes must be a multiple of 8192 and src 16-byte aligned.  A checksum (XOR of one
 * 16-byte word per lane and chunk) is XOR-ed into *checksum (device memory), so that the reads
 * cannot be optimised away; time the call with events on `stream`.
 */
int opt_gqa_debug_read_stream(const void* src, size_t bytes, unsigned* checksum, void* stream);

/*
 * Reads and clears the device status word of the current device: 0, or
 * OPT_GQA_ERR_TIMEOUT if a bounded wait inside a kernel gave up since the last
 * call.  Synchronises the device.  (Diagnostics; no counterpart in the paper.)
 */
int opt_gqa_device_status(void);

/* Human-readable name of a status code.  Never NULL. */
const char* opt_gqa_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* OPT_GQA_H_ */

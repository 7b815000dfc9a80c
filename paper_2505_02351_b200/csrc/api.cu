// extern "C" boundary of the Opt-GQA library: host-side argument checks, then one
// launcher per operation.  Nothing here allocates or keeps caller pointers; the only state of the
// library is per device: a status word on the GPU and host-side caches of addresses and attributes.
#include "common.cuh"

namespace optgqa {

// Written by kernels whose bounded waits give up; read and cleared by opt_gqa_device_status().
__device__ int g_device_status = 0;

int* device_status_ptr() {
    static std::atomic<int*> ptrs[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    int* p = ptrs[dev].load(std::memory_order_acquire);
    if (!p) {
        void* v = nullptr;
        if (cudaGetSymbolAddress(&v, g_device_status) != cudaSuccess || !v) return nullptr;
        p = static_cast<int*>(v);
        ptrs[dev].store(p, std::memory_order_release);
    }
    return p;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool dtype_ok(int dtype) { return dtype == OPT_GQA_FP32 || dtype == OPT_GQA_BF16; }
static bool shape_ok(int Hq, int Hkv, int D, int bs) {
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return false;
    const int G = Hq / Hkv;
    if (G != 1 && G != 2 && G != 4 && G != 8) return false;
    if (D != 64 && D != 128) return false;
    if (bs != 16 && bs != 32) return false;
    return true;
}

}  // namespace optgqa

using namespace optgqa;

extern "C" {

int opt_gqa_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                         const int64_t* slot_mapping, int T, int Hkv, int D, int bs, int64_t num_blocks,
                         int dtype, void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (T < 0 || Hkv <= 0 || (D != 64 && D != 128) || (bs != 16 && bs != 32) || num_blocks < 0) return OPT_GQA_ERR_SHAPE;
    if (T == 0) return OPT_GQA_OK;
    if (!k_new || !v_new || !k_cache || !v_cache || !slot_mapping) return OPT_GQA_ERR_NULL;
    if (num_blocks == 0) return OPT_GQA_ERR_SHAPE;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache)) return OPT_GQA_ERR_ALIGN;
    return launch_cache_append(k_new, v_new, k_cache, v_cache, slot_mapping, T, Hkv, D, bs, dtype,
                               static_cast<cudaStream_t>(stream));
}

static int decode_checked(bool allow_tensor_cores, int window, void* out, const void* q, const void* k_cache, const void* v_cache,
                          const int32_t* block_tables, int max_blocks_per_seq, const int32_t* context_lens,
                          const float* alibi_slopes, float scale, int B, int Hq, int Hkv, int D, int bs,
                          int64_t num_blocks, int partition_size, float* partial_out, float* partial_lse,
                          int max_partitions, int dtype, void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || !shape_ok(Hq, Hkv, D, bs) || max_blocks_per_seq < 0 || num_blocks < 0 || partition_size < 0 ||
        partition_size % 16 != 0)
        return OPT_GQA_ERR_SHAPE;
    if (B > 65535 || Hkv > 65535) return OPT_GQA_ERR_SHAPE;
    if (B == 0) return OPT_GQA_OK;
    if (!q || !k_cache || !v_cache || !block_tables || !context_lens) return OPT_GQA_ERR_NULL;
    if (num_blocks == 0 || max_blocks_per_seq == 0) return OPT_GQA_ERR_SHAPE;
    if (partition_size == 0) {
        if (!out) return OPT_GQA_ERR_NULL;
        if (!aligned16(out)) return OPT_GQA_ERR_ALIGN;
    } else {
        if (!partial_out || !partial_lse) return OPT_GQA_ERR_NULL;
        if (max_partitions <= 0 || max_partitions > 65535) return OPT_GQA_ERR_SHAPE;
        if (!aligned16(partial_out)) return OPT_GQA_ERR_ALIGN;
    }
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return OPT_GQA_ERR_ALIGN;
    int* status = device_status_ptr();
    if (!status) return OPT_GQA_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    // bf16: one CTA per (sequence, KV head, partition) -- whole partitions as work items are balanced best by the
    // hardware's own CTA scheduler (the persistent streaming kernel needs pieces smaller than a partition to balance)
    if (allow_tensor_cores && dtype == OPT_GQA_BF16)
        return launch_decode_tc(out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                                alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out,
                                partial_lse, max_partitions, status, cs);
    return launch_decode(out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens, alibi_slopes,
                         scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out, partial_lse, max_partitions,
                         window, dtype, status, cs);
}

int opt_gqa_paged_attention_decode(void* out, const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* block_tables, int max_blocks_per_seq,
                                   const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                   int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                                   float* partial_out, float* partial_lse, int max_partitions, int dtype,
                                   void* stream) {
    return decode_checked(true, 0, out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                          alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out,
                          partial_lse, max_partitions, dtype, stream);
}

int opt_gqa_paged_attention_decode_simt(void* out, const void* q, const void* k_cache, const void* v_cache,
                                        const int32_t* block_tables, int max_blocks_per_seq,
                                        const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                        int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                                        float* partial_out, float* partial_lse, int max_partitions, int dtype,
                                        void* stream) {
    return decode_checked(false, 0, out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                          alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out,
                          partial_lse, max_partitions, dtype, stream);
}

int opt_gqa_paged_attention_reduce(void* out, const float* partial_out, const float* partial_lse,
                                   const int32_t* context_lens, int B, int Hq, int D, int partition_size,
                                   int max_partitions, int dtype, void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || Hq <= 0 || (D != 64 && D != 128) || partition_size <= 0 || partition_size % 16 != 0 ||
        max_partitions <= 0)
        return OPT_GQA_ERR_SHAPE;
    if (B == 0) return OPT_GQA_OK;
    if (!out || !partial_out || !partial_lse || !context_lens) return OPT_GQA_ERR_NULL;
    if (!aligned16(out) || !aligned16(partial_out)) return OPT_GQA_ERR_ALIGN;
    return launch_reduce(out, partial_out, partial_lse, context_lens, B, Hq, D, partition_size, max_partitions, 0,
                         dtype, static_cast<cudaStream_t>(stream));
}

static int decode_balanced_checked(const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* block_tables, int max_blocks_per_seq, const int32_t* context_lens,
                                   const float* alibi_slopes, float scale, int B, int Hq, int Hkv, int D, int bs,
                                   int64_t num_blocks, int partition_size, void* workspace, size_t workspace_bytes,
                                   int max_partitions, int window, int dtype, void* stream,
                                   const FusedAppend* append = nullptr) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (dtype != OPT_GQA_BF16) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || !shape_ok(Hq, Hkv, D, bs) || max_blocks_per_seq < 0 || num_blocks < 0 || partition_size <= 0 ||
        partition_size % 16 != 0 || max_partitions <= 0 || window < 0)
        return OPT_GQA_ERR_SHAPE;
    if (B > 65535 || Hkv > 65535 || max_partitions > 65535) return OPT_GQA_ERR_SHAPE;
    if (B == 0) return OPT_GQA_OK;
    if (!q || !k_cache || !v_cache || !block_tables || !context_lens || !workspace) return OPT_GQA_ERR_NULL;
    if (num_blocks == 0 || max_blocks_per_seq == 0) return OPT_GQA_ERR_SHAPE;
    if (workspace_bytes < balanced_layout(B, Hq, Hkv, D, max_partitions).total) return OPT_GQA_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(workspace)) return OPT_GQA_ERR_ALIGN;
    int* status = device_status_ptr();
    if (!status) return OPT_GQA_ERR_CUDA;
    return launch_decode_stream(q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens, alibi_slopes,
                                scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, workspace, max_partitions, window,
                                status, static_cast<cudaStream_t>(stream), append);
}

int opt_gqa_paged_attention_decode_balanced(const void* q, const void* k_cache, const void* v_cache,
                                            const int32_t* block_tables, int max_blocks_per_seq,
                                            const int32_t* context_lens, const float* alibi_slopes, float scale,
                                            int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                                            int partition_size, void* workspace, size_t workspace_bytes,
                                            int max_partitions, int dtype, void* stream) {
    return decode_balanced_checked(q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens, alibi_slopes,
                                   scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, workspace, workspace_bytes,
                                   max_partitions, 0, dtype, stream);
}

static int reduce_balanced_checked(void* out, const void* workspace, size_t workspace_bytes,
                                   const int32_t* context_lens, int B, int Hq, int Hkv, int D, int partition_size,
                                   int max_partitions, int window, int dtype, void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (D != 64 && D != 128) || partition_size <= 0 ||
        partition_size % 16 != 0 || max_partitions <= 0 || window < 0)
        return OPT_GQA_ERR_SHAPE;
    if (B == 0) return OPT_GQA_OK;
    if (!out || !workspace || !context_lens) return OPT_GQA_ERR_NULL;
    if (workspace_bytes < balanced_layout(B, Hq, Hkv, D, max_partitions).total) return OPT_GQA_ERR_SHAPE;
    if (!aligned16(out) || !aligned16(workspace)) return OPT_GQA_ERR_ALIGN;
    return launch_reduce_balanced(out, workspace, context_lens, B, Hq, Hkv, D, partition_size, max_partitions, window,
                                  dtype, static_cast<cudaStream_t>(stream));
}

int opt_gqa_paged_attention_reduce_balanced(void* out, const void* workspace, size_t workspace_bytes,
                                            const int32_t* context_lens, int B, int Hq, int Hkv, int D,
                                            int partition_size, int max_partitions, int dtype, void* stream) {
    return reduce_balanced_checked(out, workspace, workspace_bytes, context_lens, B, Hq, Hkv, D, partition_size,
                                   max_partitions, 0, dtype, stream);
}

int opt_gqa_paged_attention_decode_local(void* out, const void* q, const void* k_cache, const void* v_cache,
                                         const int32_t* block_tables, int max_blocks_per_seq,
                                         const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                         int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                                         void* workspace, size_t workspace_bytes, int max_partitions, int window,
                                         int dtype, void* stream) {
    if (window <= 0) return OPT_GQA_ERR_SHAPE;
    if (B > 0 && !out) return OPT_GQA_ERR_NULL;
    if (dtype == OPT_GQA_FP32) {
        // fp32 caches: one partial per partition on the CUDA-core kernel (partial_out followed by partial_lse at
        // the start of the workspace), then the merge over the partitions that hold attended keys
        if (B < 0 || partition_size <= 0 || max_partitions <= 0 || Hq <= 0 || D <= 0) return OPT_GQA_ERR_SHAPE;
        if (B == 0) return OPT_GQA_OK;
        if (!workspace) return OPT_GQA_ERR_NULL;
        const size_t rows = (size_t)B * Hq * max_partitions;
        if (workspace_bytes < rows * ((size_t)D + 1) * 4) return OPT_GQA_ERR_SHAPE;
        if (!aligned16(out) || !aligned16(workspace)) return OPT_GQA_ERR_ALIGN;
        float* partial_out = static_cast<float*>(workspace);
        float* partial_lse = partial_out + rows * D;
        int rc = decode_checked(false, window, out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                                alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out,
                                partial_lse, max_partitions, dtype, stream);
        if (rc != OPT_GQA_OK) return rc;
        return launch_reduce(out, partial_out, partial_lse, context_lens, B, Hq, D, partition_size, max_partitions,
                             window, dtype, static_cast<cudaStream_t>(stream));
    }
    int rc = decode_balanced_checked(q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens, alibi_slopes,
                                     scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, workspace, workspace_bytes,
                                     max_partitions, window, dtype, stream);
    if (rc != OPT_GQA_OK || B == 0) return rc;
    return reduce_balanced_checked(out, workspace, workspace_bytes, context_lens, B, Hq, Hkv, D, partition_size,
                                   max_partitions, window, dtype, stream);
}

static int prefill_checked(bool allow_umma, int window, void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                           int max_q_len, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                           int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes,
                           float scale, int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int dtype,
                           void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (dtype != OPT_GQA_BF16) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || max_q_len < 0 || total_q_tokens < 0 || !shape_ok(Hq, Hkv, D, bs) || max_blocks_per_seq < 0 ||
        num_blocks < 0 || window < 0 || (window > 0 && !allow_umma))
        return OPT_GQA_ERR_SHAPE;
    if (B == 0 || max_q_len == 0 || total_q_tokens == 0) return OPT_GQA_OK;
    if (num_blocks == 0) return OPT_GQA_ERR_SHAPE;
    if (!out || !q || !q_start_loc || !k_cache || !v_cache || !block_tables || !context_lens) return OPT_GQA_ERR_NULL;
    if (!aligned16(out) || !aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return OPT_GQA_ERR_ALIGN;
    int* status = device_status_ptr();
    if (!status) return OPT_GQA_ERR_CUDA;
    if (allow_umma)
        return launch_prefill_umma(out, q, q_start_loc, total_q_tokens, max_q_len, k_cache, v_cache, block_tables,
                                   max_blocks_per_seq, context_lens, alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks,
                                   window, status, static_cast<cudaStream_t>(stream));
    return launch_prefill(out, q, q_start_loc, max_q_len, k_cache, v_cache, block_tables, max_blocks_per_seq,
                          context_lens, alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, status,
                          static_cast<cudaStream_t>(stream));
}

int opt_gqa_paged_attention_prefill(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                                    int max_q_len, const void* k_cache, const void* v_cache,
                                    const int32_t* block_tables, int max_blocks_per_seq, const int32_t* context_lens,
                                    const float* alibi_slopes, float scale, int B, int Hq, int Hkv, int D, int bs,
                                    int64_t num_blocks, int dtype, void* stream) {
    return prefill_checked(true, 0, out, q, q_start_loc, total_q_tokens, max_q_len, k_cache, v_cache, block_tables,
                           max_blocks_per_seq, context_lens, alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, dtype,
                           stream);
}

int opt_gqa_paged_attention_prefill_mma(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                                        int max_q_len, const void* k_cache, const void* v_cache,
                                        const int32_t* block_tables, int max_blocks_per_seq,
                                        const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                        int Hq, int Hkv, int D, int bs, int64_t num_blocks, int dtype, void* stream) {
    return prefill_checked(false, 0, out, q, q_start_loc, total_q_tokens, max_q_len, k_cache, v_cache, block_tables,
                           max_blocks_per_seq, context_lens, alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, dtype,
                           stream);
}

int opt_gqa_paged_attention_prefill_local(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens,
                                          int max_q_len, const void* k_cache, const void* v_cache,
                                          const int32_t* block_tables, int max_blocks_per_seq,
                                          const int32_t* context_lens, const float* alibi_slopes, float scale, int B,
                                          int Hq, int Hkv, int D, int bs, int64_t num_blocks, int window, int dtype,
                                          void* stream) {
    if (window <= 0) return OPT_GQA_ERR_SHAPE;
    return prefill_checked(true, window, out, q, q_start_loc, total_q_tokens, max_q_len, k_cache, v_cache, block_tables,
                           max_blocks_per_seq, context_lens, alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, dtype,
                           stream);
}

int opt_gqa_prompt_attention(void* out, const void* q, const void* k, const void* v, const int32_t* q_start_loc,
                             int total_q_tokens, int max_q_len, const float* alibi_slopes, float scale, int B, int Hq,
                             int Hkv, int D, int dtype, void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (dtype != OPT_GQA_BF16) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || max_q_len < 0 || total_q_tokens < 0 || !shape_ok(Hq, Hkv, D, 16)) return OPT_GQA_ERR_SHAPE;
    if (B == 0 || max_q_len == 0 || total_q_tokens == 0) return OPT_GQA_OK;
    if (!out || !q || !k || !v || !q_start_loc) return OPT_GQA_ERR_NULL;
    if (!aligned16(out) || !aligned16(q) || !aligned16(k) || !aligned16(v)) return OPT_GQA_ERR_ALIGN;
    int* status = device_status_ptr();
    if (!status) return OPT_GQA_ERR_CUDA;
    return launch_prompt_umma(out, q, k, v, q_start_loc, total_q_tokens, max_q_len, alibi_slopes, scale, B, Hq, Hkv, D,
                              status, static_cast<cudaStream_t>(stream));
}

// Bytes of `workspace` a decode step of these sizes uses: the balanced split's layout for bf16 caches, one
// (D + 1)-float row per (sequence, head, partition) for fp32 caches, nothing for a single pass.
static size_t step_workspace_need(int B, int Hq, int Hkv, int D, int partition_size, int max_partitions, int dtype) {
    if (partition_size <= 0 || B <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || max_partitions <= 0) return 0;
    if (dtype == OPT_GQA_BF16) return balanced_layout(B, Hq, Hkv, D, max_partitions).total;
    return (size_t)B * Hq * max_partitions * ((size_t)D + 1) * 4;
}

// Streams (sequence x KV head) up to which opt_gqa_decode_step lets the streaming kernel store the new tokens.
static constexpr long long kFusedAppendMaxStreams = 1024;

// A bf16 step whose contexts are all short and whose (sequence, KV head) streams outnumber the SMs runs as ONE launch:
// one CTA per stream walks its whole context, stores the stream's new token itself and writes out, so neither the
// slot-mapped write nor the merge is a launch of its own (on such batches the two extra launches and the pieces'
// round trip through memory cost more than the uneven finish of whole streams: 32 sequences x 8 KV heads of 512 to
// 2048 tokens measured 31 us against 36).  Only bounds known on the host decide: max_partitions * partition_size
// bounds every context.
static bool step_prefers_single_pass(int B, int Hkv, int partition_size, int max_partitions) {
    const long long streams = (long long)B * Hkv, bound = (long long)max_partitions * partition_size;
    const int sms = sm_count();
    return sms > 0 && bound <= 2048 && 2 * streams >= 3ll * sms && streams <= 4ll * sms;
}

int opt_gqa_decode_step(void* out, const void* q, const void* k_new, const void* v_new,
                        const int64_t* slot_mapping, void* k_cache, void* v_cache, const int32_t* block_tables,
                        int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes,
                        float scale, int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks,
                        int partition_size, void* workspace, size_t workspace_bytes, int max_partitions, int dtype,
                        void* stream) {
    if (!out) return B == 0 ? OPT_GQA_OK : OPT_GQA_ERR_NULL;
    if (partition_size > 0 && !workspace && B > 0) return OPT_GQA_ERR_NULL;
    if (dtype_ok(dtype) && shape_ok(Hq, Hkv, D, bs) &&
        workspace_bytes < step_workspace_need(B, Hq, Hkv, D, partition_size, max_partitions, dtype))
        return OPT_GQA_ERR_SHAPE;
    int rc;
    if (dtype == OPT_GQA_BF16 && partition_size > 0 && B > 0 && shape_ok(Hq, Hkv, D, bs) && max_partitions > 0 &&
        step_prefers_single_pass(B, Hkv, partition_size, max_partitions)) {
        if (num_blocks <= 0 || max_blocks_per_seq <= 0 || B > 65535 || partition_size % 16 != 0) return OPT_GQA_ERR_SHAPE;
        if (!q || !k_new || !v_new || !k_cache || !v_cache || !slot_mapping || !block_tables || !context_lens)
            return OPT_GQA_ERR_NULL;
        if (!aligned16(out) || !aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) ||
            !aligned16(v_cache))
            return OPT_GQA_ERR_ALIGN;
        int* status = device_status_ptr();
        if (!status) return OPT_GQA_ERR_CUDA;
        const FusedAppend fa = {k_new, v_new, k_cache, v_cache, slot_mapping};
        return launch_decode_tc(out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens, alibi_slopes,
                                scale, B, Hq, Hkv, D, bs, num_blocks, 0, nullptr, nullptr, 1, status,
                                static_cast<cudaStream_t>(stream), &fa);
    }
    if (dtype == OPT_GQA_BF16 && partition_size > 0 && B > 0) {
        // bf16 split.  With few (sequence, KV head) streams the streaming kernel stores the new tokens itself, each
        // just before the tile that holds it is fetched, and the separate launch is saved; with thousands of
        // streams those stores would stall the workers more often than the launch costs.
        const bool fuse = (long long)B * Hkv <= kFusedAppendMaxStreams;
        if (fuse) {
            // the argument checks of the slot-mapped write
            if (Hkv <= 0 || (D != 64 && D != 128) || (bs != 16 && bs != 32) || num_blocks <= 0) return OPT_GQA_ERR_SHAPE;
            if (!k_new || !v_new || !k_cache || !v_cache || !slot_mapping) return OPT_GQA_ERR_NULL;
            if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache))
                return OPT_GQA_ERR_ALIGN;
            // nothing may be enqueued if the merge's own checks would fail afterwards
            if (!aligned16(out)) return OPT_GQA_ERR_ALIGN;
        } else {
            rc = opt_gqa_cache_append(k_new, v_new, k_cache, v_cache, slot_mapping, B, Hkv, D, bs, num_blocks, dtype,
                                      stream);
            if (rc != OPT_GQA_OK) return rc;
        }
        const FusedAppend fa = {k_new, v_new, k_cache, v_cache, slot_mapping};
        rc = decode_balanced_checked(q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens, alibi_slopes,
                                     scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, workspace, workspace_bytes,
                                     max_partitions, 0, dtype, stream, fuse ? &fa : nullptr);
        if (rc != OPT_GQA_OK) return rc;
        return opt_gqa_paged_attention_reduce_balanced(out, workspace, workspace_bytes, context_lens, B, Hq, Hkv, D,
                                                       partition_size, max_partitions, dtype, stream);
    }
    // one partial per partition: partial_out [B, Hq, max_partitions, D] followed by partial_lse
    const size_t part_rows = (size_t)(B > 0 ? B : 0) * (size_t)(Hq > 0 ? Hq : 0) * (size_t)(max_partitions > 0 ? max_partitions : 0);
    rc = opt_gqa_cache_append(k_new, v_new, k_cache, v_cache, slot_mapping, B, Hkv, D, bs, num_blocks, dtype, stream);
    if (rc != OPT_GQA_OK) return rc;
    float* partial_out = static_cast<float*>(workspace);
    float* partial_lse = partial_out ? partial_out + part_rows * (size_t)(D > 0 ? D : 0) : nullptr;
    rc = opt_gqa_paged_attention_decode(out, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                                        alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size,
                                        partial_out, partial_lse, max_partitions, dtype, stream);
    if (rc != OPT_GQA_OK || partition_size == 0) return rc;
    return opt_gqa_paged_attention_reduce(out, partial_out, partial_lse, context_lens, B, Hq, D, partition_size,
                                          max_partitions, dtype, stream);
}

namespace {
// Six host arrays copied to device staging by ONE kernel that reads pinned host memory directly, in words of
// type V (16 bytes where every array allows it, else 4).  The arrays are numbered through as one range of words;
// a thread requests up to four words before it stores any, so the whole step's input crosses the bus in about one
// round trip instead of one per array.
struct HostGather {
    const void* src[6];
    void* dst[6];
    unsigned first[7];      // first[a] .. first[a + 1]: the words of array a in the joint numbering
};

extern "C++" {
template <typename V>
__global__ void __launch_bounds__(256) gather_host_kernel(const HostGather g) {
    const unsigned tid = blockIdx.x * blockDim.x + threadIdx.x, nthreads = gridDim.x * blockDim.x, total = g.first[6];
    // The words are requested from the host before the wait for the preceding kernel of the stream (the bus round
    // trip overlaps that kernel's tail); they are stored only after it, since that kernel may still read the staging
    // buffers.  This kernel never lets its own dependents start early: they read what it writes before their wait.
    bool waited = false;
    for (unsigned base = tid; base < total; base += 4 * nthreads) {
        V v[4];
        int arr[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned i = base + u * nthreads;
            arr[u] = -1;
            if (i < total) {
                int a = 0;
#pragma unroll
                for (int k = 1; k < 6; ++k) a += i >= g.first[k];
                arr[u] = a;
                v[u] = static_cast<const V*>(g.src[a])[i - g.first[a]];
            }
        }
        if (!waited) {
            grid_dependency_wait();
            waited = true;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned i = base + u * nthreads;
            if (arr[u] >= 0) static_cast<V*>(g.dst[arr[u]])[i - g.first[arr[u]]] = v[u];
        }
    }
    if (!waited) grid_dependency_wait();
}
}  // extern "C++"

// The device-side address of pinned (page-locked, mapped) host memory, or nullptr for pageable memory.
const void* device_view(const void* host) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (attr.type != cudaMemoryTypeHost || !attr.devicePointer) return nullptr;
    if (reinterpret_cast<uintptr_t>(attr.devicePointer) & 3u) return nullptr;
    return attr.devicePointer;
}

struct StagingLayout {
    size_t q, k_new, v_new, out, slots, tables, lens, total;
};
size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }
bool staging_layout(int B, int Hq, int Hkv, int D, int max_blocks, int dtype, StagingLayout* L) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || max_blocks < 0 || !dtype_ok(dtype)) return false;
    const size_t es = dtype == OPT_GQA_FP32 ? 4 : 2;
    size_t off = 0;
    L->q = off, off += round256((size_t)B * Hq * D * es);
    L->k_new = off, off += round256((size_t)B * Hkv * D * es);
    L->v_new = off, off += round256((size_t)B * Hkv * D * es);
    L->out = off, off += round256((size_t)B * Hq * D * es);
    L->slots = off, off += round256((size_t)B * sizeof(int64_t));
    L->tables = off, off += round256((size_t)B * max_blocks * sizeof(int32_t));
    L->lens = off, off += round256((size_t)B * sizeof(int32_t));
    L->total = off;
    return true;
}
}  // namespace

size_t opt_gqa_step_staging_bytes(int B, int Hq, int Hkv, int D, int max_blocks_per_seq, int dtype) {
    StagingLayout L;
    return staging_layout(B, Hq, Hkv, D, max_blocks_per_seq, dtype, &L) ? L.total : 0;
}

extern "C++" {
// The step from host buffers.  kResolved: the seven pointers are already the device-side addresses of page-locked
// memory (the caller looked them up once), so the per-call pointer queries are left out.
template <bool kResolved>
static int host_step(void* out_host, const void* q_host, const void* k_new_host, const void* v_new_host,
                     const int64_t* slot_mapping_host, const int32_t* block_tables_host,
                     const int32_t* context_lens_host, void* staging, void* k_cache, void* v_cache,
                     int max_blocks_per_seq, const float* alibi_slopes, float scale, int B, int Hq, int Hkv, int D,
                     int bs, int64_t num_blocks, int partition_size, void* workspace, size_t workspace_bytes,
                     int max_partitions, int dtype, void* stream) {
    if (!dtype_ok(dtype)) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || !shape_ok(Hq, Hkv, D, bs) || max_blocks_per_seq < 0) return OPT_GQA_ERR_SHAPE;
    if (B == 0) return OPT_GQA_OK;
    if (!out_host || !q_host || !k_new_host || !v_new_host || !slot_mapping_host || !block_tables_host ||
        !context_lens_host || !staging)
        return OPT_GQA_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(staging) & 255u) != 0) return OPT_GQA_ERR_ALIGN;
    // what the step itself would refuse is refused here, before the transfers are enqueued
    if (partition_size < 0 || partition_size % 16 != 0 || (partition_size > 0 && max_partitions <= 0) || num_blocks <= 0)
        return OPT_GQA_ERR_SHAPE;
    if (partition_size > 0 && !workspace) return OPT_GQA_ERR_NULL;
    if (!k_cache || !v_cache) return OPT_GQA_ERR_NULL;
    if (workspace_bytes < step_workspace_need(B, Hq, Hkv, D, partition_size, max_partitions, dtype)) return OPT_GQA_ERR_SHAPE;
    StagingLayout L;
    if (!staging_layout(B, Hq, Hkv, D, max_blocks_per_seq, dtype, &L)) return OPT_GQA_ERR_SHAPE;
    const size_t es = dtype == OPT_GQA_FP32 ? 4 : 2;
    char* st = static_cast<char*>(staging);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const size_t qb = (size_t)B * Hq * D * es, kb = (size_t)B * Hkv * D * es;
    // Pinned host buffers are read and written by the kernels themselves: one gather kernel instead of six copies,
    // and the last kernel of the step stores out straight into out_host.  Pageable buffers go through
    // cudaMemcpyAsync.
    const void* src[6] = {q_host, k_new_host, v_new_host, slot_mapping_host, block_tables_host, context_lens_host};
    const size_t off[6] = {L.q, L.k_new, L.v_new, L.slots, L.tables, L.lens};
    const size_t bytes[6] = {qb, kb, kb, (size_t)B * 8, (size_t)B * max_blocks_per_seq * 4, (size_t)B * 4};
    HostGather g;
    bool pinned = true, wide = true;
    for (int a = 0; a < 6; ++a) {
        const void* dv = kResolved ? src[a] : device_view(src[a]);
        pinned &= dv != nullptr && bytes[a] % 4 == 0 && (reinterpret_cast<uintptr_t>(dv) & 3u) == 0;
        wide &= bytes[a] % 16 == 0 && (reinterpret_cast<uintptr_t>(dv) & 15u) == 0;
        g.src[a] = dv;
        g.dst[a] = st + off[a];
    }
    const size_t word = wide ? 16 : 4;
    size_t words = 0;
    for (int a = 0; a < 6; ++a) {
        g.first[a] = (unsigned)words;
        words += bytes[a] / word;
    }
    pinned &= words <= 0x7fffffffull;
    g.first[6] = (unsigned)words;
    void* out_dev = !pinned ? nullptr : kResolved ? out_host : const_cast<void*>(device_view(out_host));
    pinned &= out_dev != nullptr && (reinterpret_cast<uintptr_t>(out_dev) & 15u) == 0;
    if (kResolved && !pinned) return OPT_GQA_ERR_ALIGN;     // views must be 4-byte aligned, the one of out 16-byte
    if (pinned) {
        const unsigned ctas = (unsigned)((words + 255) / 256 < 148 ? (words + 255) / 256 : 148);
        const int rc = wide ? launch_dependent(gather_host_kernel<uint4>, dim3(ctas), dim3(256), 0, cs, g)
                            : launch_dependent(gather_host_kernel<uint32_t>, dim3(ctas), dim3(256), 0, cs, g);
        if (rc != OPT_GQA_OK) return rc;
    } else {
        bool ok = true;
        for (int a = 0; a < 6; ++a)
            ok &= cudaMemcpyAsync(st + off[a], src[a], bytes[a], cudaMemcpyHostToDevice, cs) == cudaSuccess;
        if (!ok) return OPT_GQA_ERR_CUDA;
    }
    int rc = opt_gqa_decode_step(pinned ? out_dev : st + L.out, st + L.q, st + L.k_new, st + L.v_new,
                                 reinterpret_cast<const int64_t*>(st + L.slots), k_cache, v_cache,
                                 reinterpret_cast<const int32_t*>(st + L.tables), max_blocks_per_seq,
                                 reinterpret_cast<const int32_t*>(st + L.lens), alibi_slopes, scale, B, Hq, Hkv, D,
                                 bs, num_blocks, partition_size, workspace, workspace_bytes, max_partitions, dtype,
                                 stream);
    if (rc != OPT_GQA_OK) return rc;
    if (!pinned && cudaMemcpyAsync(out_host, st + L.out, qb, cudaMemcpyDeviceToHost, cs) != cudaSuccess)
        return OPT_GQA_ERR_CUDA;
    return OPT_GQA_OK;
}
}  // extern "C++"

int opt_gqa_decode_step_host(void* out_host, const void* q_host, const void* k_new_host, const void* v_new_host,
                             const int64_t* slot_mapping_host, const int32_t* block_tables_host,
                             const int32_t* context_lens_host, void* staging, void* k_cache, void* v_cache,
                             int max_blocks_per_seq, const float* alibi_slopes, float scale, int B, int Hq,
                             int Hkv, int D, int bs, int64_t num_blocks, int partition_size, void* workspace,
                             size_t workspace_bytes, int max_partitions, int dtype, void* stream) {
    return host_step<false>(out_host, q_host, k_new_host, v_new_host, slot_mapping_host, block_tables_host,
                            context_lens_host, staging, k_cache, v_cache, max_blocks_per_seq, alibi_slopes, scale, B, Hq,
                            Hkv, D, bs, num_blocks, partition_size, workspace, workspace_bytes, max_partitions, dtype,
                            stream);
}

int opt_gqa_decode_step_mapped(void* out_view, const void* q_view, const void* k_new_view, const void* v_new_view,
                               const int64_t* slot_mapping_view, const int32_t* block_tables_view,
                               const int32_t* context_lens_view, void* staging, void* k_cache, void* v_cache,
                               int max_blocks_per_seq, const float* alibi_slopes, float scale, int B, int Hq,
                               int Hkv, int D, int bs, int64_t num_blocks, int partition_size, void* workspace,
                               size_t workspace_bytes, int max_partitions, int dtype, void* stream) {
    return host_step<true>(out_view, q_view, k_new_view, v_new_view, slot_mapping_view, block_tables_view,
                           context_lens_view, staging, k_cache, v_cache, max_blocks_per_seq, alibi_slopes, scale, B, Hq,
                           Hkv, D, bs, num_blocks, partition_size, workspace, workspace_bytes, max_partitions, dtype,
                           stream);
}

size_t opt_gqa_workspace_bytes(int B, int Hq, int D, int max_partitions) {
    if (B <= 0 || Hq <= 0 || D <= 0 || max_partitions <= 0) return 0;
    // Room for either layout: one row per (sequence, head, partition), or the balanced split's pieces (the rows of
    // up to kBalancedMaxWorkers extra pieces of a group of 8 heads) with its bookkeeping.
    const size_t rows = (size_t)B * (size_t)Hq * (size_t)max_partitions + (size_t)kBalancedMaxWorkers * 8;
    return 256 + round_up_256((size_t)B * 16) + round_up_256(rows * 4) + rows * (size_t)D * 4;
}

int opt_gqa_device_status(void) {
    int* p = device_status_ptr();
    if (!p) return OPT_GQA_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, p, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return OPT_GQA_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        if (cudaMemcpy(p, &zero, sizeof zero, cudaMemcpyHostToDevice) != cudaSuccess) return OPT_GQA_ERR_CUDA;
    }
    return v;
}

const char* opt_gqa_status_string(int status) {
    switch (status) {
        case OPT_GQA_OK: return "ok";
        case OPT_GQA_ERR_NULL: return "a required pointer is NULL";
        case OPT_GQA_ERR_SHAPE: return "unsupported or inconsistent sizes";
        case OPT_GQA_ERR_DTYPE: return "unsupported dtype";
        case OPT_GQA_ERR_ALIGN: return "a data pointer is not 16-byte aligned";
        case OPT_GQA_ERR_CUDA: return "CUDA runtime error";
        case OPT_GQA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case OPT_GQA_ERR_SCRATCH: return "the call needs more scratch than the library's built-in array holds";
    }
    return "unknown status";
}

}  // extern "C"

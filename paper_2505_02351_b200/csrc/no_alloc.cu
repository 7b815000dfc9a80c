// Partitioned decode + merge for callers that cannot hand the library a workspace.
//
// Some hosts of this library have no way to allocate device memory at the point where they call it: a
// plugin running inside a serving engine that has already claimed the whole GPU for its cache pool, a
// callback invoked from a context where cudaMalloc would synchronise the device or is simply forbidden
// by the embedding runtime.  The partitioned decode needs scratch for the partitions' partial results;
// this file keeps that scratch in a fixed array that is part of the loaded module, so the call needs
// nothing beyond the caller's inputs and outputs.
//
// The array belongs to the module: every GPU on which the library is used holds its 8 MiB from the
// first call until the process exits, and every call on that GPU shares it.  Calls whose kernels can
// overlap on the GPU (different streams) therefore race on it; issue them on one stream, or order them.
// Nothing in it has to be cleared between calls: the merge reads exactly the entries (sequence, head,
// partition < ceil(n / P)) that the decode kernel of the same call wrote, never what an earlier call left.
#include "common.cuh"

namespace optgqa {
namespace {

constexpr size_t kScratchFloats = OPT_GQA_STATIC_SCRATCH_BYTES / sizeof(float);

// In host code this name is only a handle for the runtime; the device address comes from
// cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_scratch[kScratchFloats];

// Device address of the array on the current device, resolved once per device (with that device current; the
// stream passed to the entry point must belong to that device).  The cache is atomic: host threads that make their
// first call together each look the address up and store the same value.
float* static_scratch_ptr() {
    static std::atomic<float*> ptrs[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    float* p = ptrs[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess || !p) return nullptr;
        ptrs[dev].store(p, std::memory_order_release);
    }
    return p;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace optgqa

using namespace optgqa;

extern "C" int opt_gqa_paged_attention_decode_no_alloc(void* out, const void* q, const void* k_cache,
                                                       const void* v_cache, const int32_t* block_tables,
                                                       int max_blocks_per_seq, const int32_t* context_lens,
                                                       const float* alibi_slopes, float scale, int B, int Hq,
                                                       int Hkv, int D, int bs, int64_t num_blocks,
                                                       int partition_size, int max_partitions, int dtype,
                                                       void* stream) {
    if (dtype != OPT_GQA_FP32 && dtype != OPT_GQA_BF16) return OPT_GQA_ERR_DTYPE;
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (D != 64 && D != 128) || (bs != 16 && bs != 32) ||
        max_blocks_per_seq < 0 || (B > 0 && max_blocks_per_seq == 0) || num_blocks < 0 || partition_size <= 0 || partition_size % 16 != 0 ||
        max_partitions <= 0)
        return OPT_GQA_ERR_SHAPE;
    const int G = Hq / Hkv;
    if (G != 1 && G != 2 && G != 4 && G != 8) return OPT_GQA_ERR_SHAPE;
    if (B > 65535 || Hkv > 65535 || max_partitions > 65535) return OPT_GQA_ERR_SHAPE;
    if (B == 0) return OPT_GQA_OK;
    if (!out || !q || !k_cache || !v_cache || !block_tables || !context_lens) return OPT_GQA_ERR_NULL;
    if (num_blocks == 0) return OPT_GQA_ERR_SHAPE;
    if (!aligned16(out) || !aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache)) return OPT_GQA_ERR_ALIGN;
    // partial_out [B, Hq, max_partitions, D] followed by partial_lse [B, Hq, max_partitions]
    const unsigned long long rows = (unsigned long long)B * Hq * max_partitions;
    if (rows * (unsigned long long)(D + 1) > kScratchFloats) return OPT_GQA_ERR_SCRATCH;
    float* scratch = static_scratch_ptr();
    int* status = device_status_ptr();
    if (!scratch || !status) return OPT_GQA_ERR_CUDA;
    float* partial_out = scratch;
    float* partial_lse = scratch + rows * D;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    int rc;
    if (dtype == OPT_GQA_BF16)
        rc = launch_decode_tc(nullptr, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                              alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out,
                              partial_lse, max_partitions, status, cs);
    else
        rc = launch_decode(nullptr, q, k_cache, v_cache, block_tables, max_blocks_per_seq, context_lens,
                           alibi_slopes, scale, B, Hq, Hkv, D, bs, num_blocks, partition_size, partial_out,
                           partial_lse, max_partitions, 0, dtype, status, cs);
    if (rc != OPT_GQA_OK) return rc;
    return launch_reduce(out, partial_out, partial_lse, context_lens, B, Hq, D, partition_size, max_partitions, 0,
                         dtype, cs);
}

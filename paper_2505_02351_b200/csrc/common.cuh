// Shared device helpers of the Opt-GQA CUDA library (sm_100a): PTX wrappers for
// mbarriers and bulk async copies, storage-type unpacking, launch plumbing.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "opt_gqa.h"

namespace optgqa {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ----------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

// Makes freshly initialised barriers visible to the async proxy.
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Orders earlier generic-proxy accesses to shared memory before later async-proxy ones.
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Bounded wait: gives up after about kWaitLimitCycles SM clocks (~0.14 s; real waits last microseconds), records
// the timeout and returns false.  The bound is on elapsed time, not on the number of polls: one try_wait may
// itself block for a while before it reports failure.
constexpr long long kWaitLimitCycles = 1ll << 28;
// try_wait that lets the hardware park the warp for up to `ns` nanoseconds while the phase is pending, so that a
// waiting warp does not take issue slots from the warps it is waiting for.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
        : "memory");
    return done != 0;
}

__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status,
                                          long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long start = clock64();
    do {
        if (mbar_try_wait_parked(bar, parity, 4000)) return true;
    } while (clock64() - start < limit_cycles);
    atomicExch(status, OPT_GQA_ERR_TIMEOUT);
    return false;
}

// 1-D bulk copy global -> this CTA's shared memory, completion counted on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// The same copy with an L2 cache policy (createpolicy).
__device__ __forceinline__ void bulk_g2s_hint(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// L2 policy for data that is read once: its lines are the first to be evicted.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Programmatic dependent launch: wait for the grid this one depends on / let dependents start.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch that may begin while the preceding kernel of the stream is still draining (programmatic
// stream serialisation).  The kernel must execute grid_dependency_wait() before it touches anything
// the preceding kernel writes; with a predecessor that never signals, this is an ordinary launch.
template <typename... KArgs, typename... Args>
inline int launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                            Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) == cudaSuccess ? OPT_GQA_OK : OPT_GQA_ERR_CUDA;
}

// ----------------------------------------------------------------------------- storage types
// Two adjacent bf16 values packed in one 32-bit word -> (low element, high element) as fp32.
__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

__device__ __forceinline__ uint32_t float2_to_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <typename T>
struct Store;
template <>
struct Store<float> {
    static constexpr int kDtype = OPT_GQA_FP32;
};
template <>
struct Store<__nv_bfloat16> {
    static constexpr int kDtype = OPT_GQA_BF16;
};

// Address of the current device's status word (api.cu); nullptr if the runtime refuses.
int* device_status_ptr();

// Multiprocessors of the current device (cached per device); 0 if the runtime refuses (decode_stream.cu).
int sm_count();

// Per-device host-side caches (symbol addresses, attribute flags, SM counts) are arrays of atomics indexed by the
// device ordinal: two host threads making their first call together both do the (idempotent) set-up and store the
// same value, without a data race.
constexpr int kMaxDevices = 64;

// Raises the dynamic shared memory limit of `kernel` once per device.  `done` is the launcher's own
// `static std::atomic<bool> [kMaxDevices]`.
template <typename Kernel>
inline bool ensure_smem_limit(Kernel kernel, int bytes, std::atomic<bool>* done) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached && done[dev].load(std::memory_order_acquire)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (cached) done[dev].store(true, std::memory_order_release);
    return true;
}

// ----------------------------------------------------------------------------- host-side launchers (one per .cu)
int launch_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                        const int64_t* slot_mapping, int T, int Hkv, int D, int bs, int dtype,
                        cudaStream_t stream);

int launch_decode(void* out, const void* q, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                  int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes, float scale,
                  int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size, float* partial_out,
                  float* partial_lse, int max_partitions, int window, int dtype, int* device_status,
                  cudaStream_t stream);

// Workspace of the balanced split (bf16 caches, partition_size > 0).  The stream of 16-token tiles
// (sequence, KV head, partition order) is cut into one range per worker at TILE granularity; a piece is the
// part of one partition inside one range, and piece (partition index i in that order, worker w) owns rows
// (i + w) * G .. + G - 1 of partial_lse / partial_out.  header = {tiles in the stream, workers};
// seq_info[s] = {tiles, partitions} of one head summed over the sequences before s.
constexpr int kBalancedMaxWorkers = 2048;
struct BalancedLayout {
    size_t header, seq_info, lse, out, total;
    unsigned long long rows;      // rows of partial_lse / partial_out
};
inline size_t round_up_256(size_t x) { return (x + 255) & ~(size_t)255; }
inline BalancedLayout balanced_layout(int B, int Hq, int Hkv, int D, int max_partitions) {
    BalancedLayout L;
    const unsigned long long G = (unsigned long long)(Hq / Hkv);
    L.rows = ((unsigned long long)B * Hkv * max_partitions + kBalancedMaxWorkers) * G;
    L.header = 0;
    L.seq_info = 256;
    L.lse = L.seq_info + round_up_256((size_t)B * 16);
    L.out = L.lse + round_up_256((size_t)L.rows * 4);
    L.total = L.out + (size_t)L.rows * D * 4;
    return L;
}

// The step's new K/V rows for the streaming kernel to store itself (Algorithm 2, "Store reshaped K, V into C_K,
// C_V"): the worker that is about to fetch the tile holding a sequence's last position first writes that sequence's
// new token to its slot, which saves the separate launch of the slot-mapped write.
struct FusedAppend {
    const void* k_new;              // [B, Hkv, D] bf16
    const void* v_new;
    void* k_cache;
    void* v_cache;
    const int64_t* slot_mapping;    // [B]; negative: nothing to store
};

// bf16 only: the query group as rows of tensor-core tiles (decode_tc.cu).  append != nullptr: see FusedAppend.
int launch_decode_tc(void* out, const void* q, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                     int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes, float scale,
                     int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                     float* partial_out, float* partial_lse, int max_partitions, int* device_status,
                     cudaStream_t stream, const FusedAppend* append = nullptr);

// bf16, partition_size > 0, balanced split into `workspace`: persistent streaming kernel, one worker per warp
// (decode_stream.cu).  append != nullptr: see FusedAppend.
int launch_decode_stream(const void* q, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                         int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes, float scale,
                         int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                         void* workspace, int max_partitions, int window, int* device_status, cudaStream_t stream,
                         const FusedAppend* append = nullptr);

// Workers (warps) of the grid that launch_decode_stream uses for the balanced split of these sizes on the current
// device; 0 if the device cannot be queried.
long long stream_grid_workers(int B, int Hkv, int max_partitions, int partition_size);

// Merge of the balanced split's pieces (reduce.cu).
int launch_reduce_balanced(void* out, const void* workspace, const int32_t* context_lens, int B, int Hq, int Hkv,
                           int D, int partition_size, int max_partitions, int window, int dtype, cudaStream_t stream);

// window > 0: the partitions that lie wholly before a sequence's last `window` keys were not written and are skipped.
int launch_reduce(void* out, const float* partial_out, const float* partial_lse, const int32_t* context_lens,
                  int B, int Hq, int D, int partition_size, int max_partitions, int window, int dtype,
                  cudaStream_t stream);

int launch_prefill(void* out, const void* q, const int32_t* q_start_loc, int max_q_len, const void* k_cache,
                   const void* v_cache, const int32_t* block_tables, int max_blocks_per_seq,
                   const int32_t* context_lens, const float* alibi_slopes, float scale, int B, int Hq, int Hkv,
                   int D, int bs, int64_t num_blocks, int* device_status, cudaStream_t stream);

// bf16, any scale: tcgen05.mma with accumulators in tensor memory (prefill_umma.cu).
int launch_prefill_umma(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens, int max_q_len,
                        const void* k_cache, const void* v_cache, const int32_t* block_tables, int max_blocks_per_seq,
                        const int32_t* context_lens, const float* alibi_slopes, float scale, int B, int Hq, int Hkv,
                        int D, int bs, int64_t num_blocks, int window, int* device_status, cudaStream_t stream);

// bf16: the prompt branch with empty caches (contiguous k, v of the new tokens), same kernel.
int launch_prompt_umma(void* out, const void* q, const void* k, const void* v, const int32_t* q_start_loc,
                       int total_q_tokens, int max_q_len, const float* alibi_slopes, float scale, int B, int Hq,
                       int Hkv, int D, int* device_status, cudaStream_t stream);

}  // namespace optgqa

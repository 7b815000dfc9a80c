// Diagnostics of the Opt-GQA library (no counterpart in the paper): a read-only streaming probe that
// shows what the decode kernels' data path can reach on this GPU when no arithmetic is attached to it,
// and a kernel whose bounded wait runs out on purpose, so that a host can test its handling of
// OPT_GQA_ERR_TIMEOUT without a fault or a hang.
#include "common.cuh"

namespace optgqa {
namespace {

constexpr int kProbeWarps = 4;          // workers per CTA, as in the streaming decode kernel
constexpr int kProbeStages = 2;         // ring depth per worker
constexpr int kProbeCtasPerSm = 2;
constexpr int kProbeChunk = 8192;       // bytes per ring stage: a K tile plus a V tile of 16 tokens x 128 dims, bf16
constexpr int kProbeSmem = kProbeWarps * kProbeStages * (kProbeChunk + 8);

// Every warp streams chunks me, me + workers, ... of `src` through a private two-stage ring of bulk async
// copies (read-once L2 policy) and folds one 16-byte word per lane and chunk into a checksum.  The ring shape,
// the copy engine and the number of bytes in flight are those of the streaming decode kernel.
__global__ void __launch_bounds__(kProbeWarps * 32, kProbeCtasPerSm)
read_probe_kernel(const char* __restrict__ src, long long chunks, unsigned* __restrict__ checksum, int* status) {
    extern __shared__ __align__(128) char probe_smem[];
    char (*ring)[kProbeStages][kProbeChunk] = reinterpret_cast<char (*)[kProbeStages][kProbeChunk]>(probe_smem);
    uint64_t (*bars)[kProbeStages] =
        reinterpret_cast<uint64_t (*)[kProbeStages]>(probe_smem + kProbeWarps * kProbeStages * kProbeChunk);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long workers = (long long)gridDim.x * kProbeWarps, me = (long long)blockIdx.x * kProbeWarps + warp;
    const uint64_t read_once = l2_policy_evict_first();
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kProbeStages; ++i) mbar_init(&bars[warp][i], 1);
        fence_barrier_init();
    }
    __syncwarp();
    const long long cnt = chunks > me ? (chunks - me + workers - 1) / workers : 0;
    auto issue = [&](long long k) {
        if (lane == 0) {
            const int st = (int)(k % kProbeStages);
            mbar_expect_tx(&bars[warp][st], kProbeChunk);
            bulk_g2s_hint(ring[warp][st], src + (me + k * workers) * kProbeChunk, kProbeChunk, &bars[warp][st], read_once);
        }
    };
    for (long long k = 0; k < kProbeStages && k < cnt; ++k) issue(k);
    uint4 acc = make_uint4(0, 0, 0, 0);
    long long k = 0;
    bool ok = true;
    for (; k < cnt; ++k) {
        const int st = (int)(k % kProbeStages);
        ok = __all_sync(0xffffffffu, mbar_wait(&bars[warp][st], (uint32_t)((k / kProbeStages) & 1), status));
        if (!ok) break;
        const uint4 w = *reinterpret_cast<const uint4*>(ring[warp][st] + lane * 256);
        acc.x ^= w.x;
        acc.y ^= w.y;
        acc.z ^= w.z;
        acc.w ^= w.w;
        __syncwarp();
        if (k + kProbeStages < cnt) issue(k + kProbeStages);
    }
    if (!ok)    // a wait gave up (recorded): give the copies in flight a bounded chance to land before the CTA ends
        for (long long kk = k; kk < cnt && kk < k + kProbeStages; ++kk)
            mbar_wait(&bars[warp][kk % kProbeStages], (uint32_t)((kk / kProbeStages) & 1), status);
    unsigned x = acc.x ^ acc.y ^ acc.z ^ acc.w;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) x ^= __shfl_xor_sync(0xffffffffu, x, o);
    if (lane == 0 && cnt > 0) atomicXor(checksum, x);
}

// One warp arms an mbarrier for bytes that nothing will ever send and waits on it with the given limit: the
// wait runs out, records OPT_GQA_ERR_TIMEOUT in the status word and the kernel returns.
__global__ void __launch_bounds__(32) wait_timeout_probe_kernel(int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_barrier_init();
        mbar_expect_tx(&bar, 16);
    }
    __syncwarp();
    mbar_wait(&bar, 0, status, limit_cycles);
}

}  // namespace
}  // namespace optgqa

using namespace optgqa;

extern "C" int opt_gqa_debug_read_stream(const void* src, size_t bytes, unsigned* checksum, void* stream) {
    if (bytes == 0) return OPT_GQA_OK;
    if (!src || !checksum) return OPT_GQA_ERR_NULL;
    if (bytes % kProbeChunk != 0) return OPT_GQA_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(src) & 15u) return OPT_GQA_ERR_ALIGN;
    int* status = device_status_ptr();
    int dev = 0, sms = 0;
    if (!status || cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return OPT_GQA_ERR_CUDA;
    const long long chunks = (long long)(bytes / kProbeChunk);
    long long ctas = (chunks + kProbeWarps - 1) / kProbeWarps;
    if (ctas > (long long)sms * kProbeCtasPerSm) ctas = (long long)sms * kProbeCtasPerSm;
    static std::atomic<bool> configured[kMaxDevices];
    if (!ensure_smem_limit(read_probe_kernel, kProbeSmem, configured)) return OPT_GQA_ERR_CUDA;
    read_probe_kernel<<<(unsigned)ctas, kProbeWarps * 32, kProbeSmem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const char*>(src), chunks, checksum, status);
    return cudaGetLastError() == cudaSuccess ? OPT_GQA_OK : OPT_GQA_ERR_CUDA;
}

extern "C" int opt_gqa_debug_wait_timeout(long long limit_cycles, void* stream) {
    if (limit_cycles < 1 || limit_cycles > (1ll << 24)) return OPT_GQA_ERR_SHAPE;
    int* status = device_status_ptr();
    if (!status) return OPT_GQA_ERR_CUDA;
    wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, limit_cycles);
    return cudaGetLastError() == cudaSuccess ? OPT_GQA_OK : OPT_GQA_ERR_CUDA;
}

// Slot-mapped write of new K/V rows into the paged cache (Algorithm 1, "Reshape
// and store K, V into C_K, C_V"; Eq. 2).  A pure copy: one thread moves 16 bytes
// of K and 16 bytes of V, so a (token, kv head) row is written by consecutive
// lanes as one coalesced segment.
#include "common.cuh"

namespace optgqa {

// row_vecs = D * element_size / 16: 16-byte vectors per (token, head) row.
__global__ void __launch_bounds__(256)
cache_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* __restrict__ k_cache,
                    uint4* __restrict__ v_cache, const int64_t* __restrict__ slot_mapping, long long total_vecs,
                    int Hkv, int row_vecs, int bs) {
    grid_dependency_launch();   // the attention grid may start its prologue; it waits before reading the cache
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total_vecs) return;
    int vec = (int)(i % row_vecs);
    long long th = i / row_vecs;  // token * Hkv + head
    int h = (int)(th % Hkv);
    long long t = th / Hkv;
    grid_dependency_wait();     // the new rows and the slots may come from the preceding grid, which may also still read the cache
    long long slot = slot_mapping[t];
    if (slot < 0) return;
    long long page = slot / bs;
    int off = (int)(slot % bs);
    long long dst = (((page * Hkv + h) * bs) + off) * row_vecs + vec;
    k_cache[dst] = k_new[i];
    v_cache[dst] = v_new[i];
}

int launch_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                        const int64_t* slot_mapping, int T, int Hkv, int D, int bs, int dtype,
                        cudaStream_t stream) {
    const int es = dtype == OPT_GQA_FP32 ? 4 : 2;
    const int row_vecs = D * es / 16;
    const long long total = (long long)T * Hkv * row_vecs;
    const int threads = 256;
    const long long blocks = (total + threads - 1) / threads;
    // launched while the preceding grid drains; the kernel waits for it before it touches memory
    return launch_dependent(cache_append_kernel, dim3((unsigned)blocks), dim3(threads), 0, stream,
                            static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                            static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache), slot_mapping, total, Hkv,
                            row_vecs, bs);
}

}  // namespace optgqa

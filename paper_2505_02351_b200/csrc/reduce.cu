// Log-sum-exp merge of the context partitions (the paragraph before Eq. 1: each
// partition's output is kept and then combined into the sequence's result):
//   out = sum_p e^{lse_p - L} o_p / sum_p e^{lse_p - L},  L = max_p lse_p,  p < ceil(n_s / P).
// One CTA per (sequence, query head).  A lane owns D/32 adjacent output columns, so a
// warp reads one partial row as one coalesced segment; the warps of the CTA take the
// partitions round-robin (independent loads in flight instead of one dependent chain
// over all partitions) and are folded through shared memory at the end.
#include "common.cuh"

namespace optgqa {

constexpr int kReduceWarps = 4;

template <typename T, int D>
__global__ void __launch_bounds__(kReduceWarps * 32)
reduce_kernel(T* __restrict__ out, const float* __restrict__ partial_out, const float* __restrict__ partial_lse,
              const int32_t* __restrict__ context_lens, int Hq, int partition_size, int max_partitions) {
    constexpr int V = D / 32;             // columns per lane
    __shared__ float s_num[kReduceWarps][D];
    __shared__ float s_den[kReduceWarps];
    grid_dependency_launch();
    const int row = blockIdx.x;            // s * Hq + h
    const int s = row / Hq;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = context_lens[s];         // an input of the step, not produced by the decode grid
    const int np = (n + partition_size - 1) / partition_size;
    T* o = out + (size_t)row * D;
    if (np <= 0) {
        for (int d = threadIdx.x; d < D; d += blockDim.x) o[d] = T(0.f);
        return;
    }
    grid_dependency_wait();                // the partials come from the decode grid
    const float* lse = partial_lse + (size_t)row * max_partitions;
    const float* po = partial_out + (size_t)row * max_partitions * D + lane * V;

    float L = -INFINITY;
    for (int p = lane; p < np; p += 32) L = fmaxf(L, lse[p]);
#pragma unroll
    for (int o2 = 16; o2 >= 1; o2 >>= 1) L = fmaxf(L, __shfl_xor_sync(0xffffffffu, L, o2));

    float num[V];
#pragma unroll
    for (int v = 0; v < V; ++v) num[v] = 0.f;
    float den = 0.f;
#pragma unroll 4
    for (int p = warp; p < np; p += kReduceWarps) {
        const float w = ex2((lse[p] - L) * kLog2e);
        den += w;
        if constexpr (V == 4) {
            const float4 x = *reinterpret_cast<const float4*>(po + (size_t)p * D);
            num[0] = fmaf(w, x.x, num[0]);
            num[1] = fmaf(w, x.y, num[1]);
            num[2] = fmaf(w, x.z, num[2]);
            num[3] = fmaf(w, x.w, num[3]);
        } else {
            const float2 x = *reinterpret_cast<const float2*>(po + (size_t)p * D);
            num[0] = fmaf(w, x.x, num[0]);
            num[1] = fmaf(w, x.y, num[1]);
        }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) s_num[warp][lane * V + v] = num[v];
    if (lane == 0) s_den[warp] = den;
    __syncthreads();
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int w = 0; w < kReduceWarps; ++w) {
            a += s_num[w][d];
            b += s_den[w];
        }
        const float r = a / b;
        if constexpr (sizeof(T) == 2) o[d] = __float2bfloat16_rn(r);
        else o[d] = r;
    }
}

template <typename T, int D>
static int launch_reduce_t(void* out, const float* partial_out, const float* partial_lse,
                           const int32_t* context_lens, int B, int Hq, int partition_size, int max_partitions,
                           cudaStream_t stream) {
    return launch_dependent(reduce_kernel<T, D>, dim3((unsigned)B * (unsigned)Hq), dim3(kReduceWarps * 32), 0, stream,
                            static_cast<T*>(out), partial_out, partial_lse, context_lens, Hq, partition_size,
                            max_partitions);
}

int launch_reduce(void* out, const float* partial_out, const float* partial_lse, const int32_t* context_lens,
                  int B, int Hq, int D, int partition_size, int max_partitions, int dtype, cudaStream_t stream) {
    if (dtype == OPT_GQA_BF16) {
        if (D == 128)
            return launch_reduce_t<__nv_bfloat16, 128>(out, partial_out, partial_lse, context_lens, B, Hq,
                                                       partition_size, max_partitions, stream);
        return launch_reduce_t<__nv_bfloat16, 64>(out, partial_out, partial_lse, context_lens, B, Hq, partition_size,
                                                  max_partitions, stream);
    }
    if (D == 128)
        return launch_reduce_t<float, 128>(out, partial_out, partial_lse, context_lens, B, Hq, partition_size,
                                           max_partitions, stream);
    return launch_reduce_t<float, 64>(out, partial_out, partial_lse, context_lens, B, Hq, partition_size,
                                      max_partitions, stream);
}

}  // namespace optgqa

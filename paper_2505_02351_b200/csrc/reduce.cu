// Log-sum-exp merge of the context partitions (the paragraph before Eq. 1: the
// per-block outputs are kept and combined into the sequence's result):
//   out = sum_p e^{lse_p - L} o_p / sum_p e^{lse_p - L},  L = max_p lse_p,  p < ceil(n_s / P).
// One CTA of D threads per (sequence, query head); thread d owns output column d,
// so every partial row is read as one coalesced segment.
#include "common.cuh"

namespace optgqa {

template <typename T>
__global__ void reduce_kernel(T* __restrict__ out, const float* __restrict__ partial_out,
                              const float* __restrict__ partial_lse, const int32_t* __restrict__ context_lens,
                              int Hq, int D, int partition_size, int max_partitions) {
    grid_dependency_wait();   // no-op unless launched as a programmatic dependent of the decode grid
    const int row = blockIdx.x;            // s * Hq + h
    const int s = row / Hq;
    const int d = threadIdx.x;
    const int n = context_lens[s];
    const int np = (n + partition_size - 1) / partition_size;
    T* o = out + (size_t)row * D + d;
    if (np <= 0) {
        *o = T(0.f);
        return;
    }
    const float* lse = partial_lse + (size_t)row * max_partitions;
    const float* po = partial_out + (size_t)row * max_partitions * D + d;
    float L = -INFINITY;
    for (int p = 0; p < np; ++p) L = fmaxf(L, lse[p]);
    float num = 0.f, den = 0.f;
#pragma unroll 4
    for (int p = 0; p < np; ++p) {
        const float w = ex2((lse[p] - L) * kLog2e);
        den += w;
        num = fmaf(w, po[(size_t)p * D], num);
    }
    const float r = num / den;
    if constexpr (sizeof(T) == 2) *o = __float2bfloat16_rn(r);
    else *o = r;
}

int launch_reduce(void* out, const float* partial_out, const float* partial_lse, const int32_t* context_lens,
                  int B, int Hq, int D, int partition_size, int max_partitions, int dtype, cudaStream_t stream) {
    const unsigned rows = (unsigned)B * (unsigned)Hq;
    if (dtype == OPT_GQA_BF16)
        reduce_kernel<__nv_bfloat16><<<rows, D, 0, stream>>>(static_cast<__nv_bfloat16*>(out), partial_out,
                                                            partial_lse, context_lens, Hq, D, partition_size,
                                                            max_partitions);
    else
        reduce_kernel<float><<<rows, D, 0, stream>>>(static_cast<float*>(out), partial_out, partial_lse,
                                                    context_lens, Hq, D, partition_size, max_partitions);
    return cudaGetLastError() == cudaSuccess ? OPT_GQA_OK : OPT_GQA_ERR_CUDA;
}

}  // namespace optgqa

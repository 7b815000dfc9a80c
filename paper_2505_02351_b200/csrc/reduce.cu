// Log-sum-exp merge of the context partitions (the paragraph before Eq. 1: each
// partition's output is kept and then combined into the sequence's result):
//   out = sum_p e^{lse_p - L} o_p / sum_p e^{lse_p - L},  L = max_p lse_p,  p < ceil(n_s / P).
// One CTA per (sequence, query head).  A lane owns D/32 adjacent output columns, so a
// warp reads one partial row as one coalesced segment; the warps of the CTA take the
// partitions round-robin and are folded through shared memory at the end.  The first
// kReducePre rows of every warp's share are requested together with the log-sum-exps,
// before the maximum is known (with up to 64 partitions that is all of them: the merge
// is one round trip to memory, not two dependent ones).
#include <type_traits>

#include "common.cuh"

namespace optgqa {

constexpr int kReduceWarps = 8;
constexpr int kReducePre = 8;

template <typename T, int D>
__global__ void __launch_bounds__(kReduceWarps * 32)
reduce_kernel(T* __restrict__ out, const float* __restrict__ partial_out, const float* __restrict__ partial_lse,
              const int32_t* __restrict__ context_lens, int Hq, int partition_size, int max_partitions, int window) {
    constexpr int V = D / 32;             // columns per lane
    using Vec = typename std::conditional<V == 4, float4, float2>::type;
    __shared__ float s_num[kReduceWarps][D];
    __shared__ float s_den[kReduceWarps];
    grid_dependency_launch();
    const int row = blockIdx.x;            // s * Hq + h
    const int s = row / Hq;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = context_lens[s];         // an input of the step, not produced by the decode grid
    // never beyond the rows the decode grid had (max_partitions is the caller's promise; a length that breaks it gives
    // a wrong row, not a read past the partials)
    const int np = min((n + partition_size - 1) / partition_size, max_partitions);
    // with a local mask the partitions wholly before the first attended key hold nothing
    const int p_lo = window > 0 ? max(0, n - window) / partition_size : 0;
    T* o = out + (size_t)row * D;
    grid_dependency_wait();                // the partials come from the decode grid; out may still be read by its last user
    if (np <= p_lo) {
        for (int d = threadIdx.x; d < D; d += blockDim.x) o[d] = T(0.f);
        return;
    }
    const float* lse = partial_lse + (size_t)row * max_partitions;
    const float* po = partial_out + (size_t)row * max_partitions * D + lane * V;

    float lpre[kReducePre];
    Vec xpre[kReducePre];
#pragma unroll
    for (int k = 0; k < kReducePre; ++k) {
        const int p = p_lo + warp + k * kReduceWarps;
        lpre[k] = -INFINITY;
        if (p < np) {
            lpre[k] = lse[p];
            xpre[k] = *reinterpret_cast<const Vec*>(po + (size_t)p * D);
        }
    }
    float L = -INFINITY;
    for (int p = p_lo + lane; p < np; p += 32) L = fmaxf(L, lse[p]);
#pragma unroll
    for (int o2 = 16; o2 >= 1; o2 >>= 1) L = fmaxf(L, __shfl_xor_sync(0xffffffffu, L, o2));

    float num[V];
#pragma unroll
    for (int v = 0; v < V; ++v) num[v] = 0.f;
    float den = 0.f;
    auto add_row = [&](float l, Vec x) {
        const float w = ex2((l - L) * kLog2e);
        den += w;
        num[0] = fmaf(w, x.x, num[0]);
        num[1] = fmaf(w, x.y, num[1]);
        if constexpr (V == 4) {
            num[2] = fmaf(w, x.z, num[2]);
            num[3] = fmaf(w, x.w, num[3]);
        }
    };
#pragma unroll
    for (int k = 0; k < kReducePre; ++k)
        if (p_lo + warp + k * kReduceWarps < np) add_row(lpre[k], xpre[k]);
#pragma unroll 4
    for (int p = p_lo + warp + kReducePre * kReduceWarps; p < np; p += kReduceWarps)
        add_row(lse[p], *reinterpret_cast<const Vec*>(po + (size_t)p * D));
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

// The same merge over the pieces of the balanced split (see balanced_layout).  The pieces of the row's
// (sequence, KV head) stream carry consecutive numbers -- (partition index) + (worker index), and from one piece
// to the next exactly one of the two grows, or both, in which case the decode kernel marked the number in between
// with lse = -inf -- so the merge is one sweep over rows r0 .. r1 of partial_lse / partial_out: r0 belongs to the
// stream's first tile, r1 to its last.  All loads of the sweep are independent.
// A CTA has 8 warps and merges 8 / WPR rows, WPR warps per row (chosen by the launcher from the number of
// rows, so that batches of many short sequences do not pay for warps with nothing to sweep).
constexpr int kBalWarps = 8;

template <typename T, int D, int WPR, int kPre>
__global__ void __launch_bounds__(kBalWarps * 32)
reduce_balanced_kernel(T* __restrict__ out, const float* __restrict__ partial_out,
                       const float* __restrict__ partial_lse, const long long* __restrict__ header,
                       const long long* __restrict__ seq_info, const int32_t* __restrict__ context_lens, int rows,
                       int Hq, int Hkv, int partition_size, int window, int B, long long grid_workers) {
    constexpr int V = D / 32;             // columns per lane
    constexpr int RPB = kBalWarps / WPR;  // rows per CTA
    __shared__ float s_num[kBalWarps][D];
    __shared__ float s_den[kBalWarps];
    __shared__ float s_max[kBalWarps];
    grid_dependency_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rib = warp / WPR, sub = warp % WPR;
    const int row = blockIdx.x * RPB + rib;                 // s * Hq + h
    const bool active = row < rows;
    const int s = active ? row / Hq : 0, h = active ? row % Hq : 0, G = Hq / Hkv, kvh = h / G, hh = h % G;
    const int n = active ? context_lens[s] : 0;             // an input of the step, not produced by the decode grid
    // the sequence's stream starts at the tile of its first attended key; partitions are counted from there
    const int P16 = partition_size / 16;
    const int tiles = (n + 15) / 16 - (window > 0 ? max(0, n - window) / 16 : 0);
    const int np = (tiles + P16 - 1) / P16;
    // With at most 32 sequences a warp works out the decode grid's bookkeeping (tiles and partitions before the
    // sequence, tiles in all, ranges) from the lengths itself, while the decode grid is still running, instead of
    // reading it from the workspace afterwards: one dependent round trip less between the two grids.
    const bool own_counts = grid_workers > 0 && B <= 32;
    long long total = 0, workers = 1, tiles_before = 0, parts_before = 0;
    if (own_counts) {
        const int nl = lane < B ? context_lens[lane] : 0;
        const int tl = (nl + 15) / 16 - (window > 0 ? max(0, nl - window) / 16 : 0);
        int it = tl, ip = (tl + P16 - 1) / P16;
#pragma unroll
        for (int o2 = 1; o2 < 32; o2 <<= 1) {
            const int vt = __shfl_up_sync(0xffffffffu, it, o2), vp = __shfl_up_sync(0xffffffffu, ip, o2);
            if (lane >= o2) {
                it += vt;
                ip += vp;
            }
        }
        total = (long long)__shfl_sync(0xffffffffu, it, 31) * Hkv;
        tiles_before = __shfl_sync(0xffffffffu, it, s) - tiles;
        parts_before = __shfl_sync(0xffffffffu, ip, s) - np;
        workers = total < grid_workers ? (total > 0 ? total : 1) : grid_workers;
    }
    grid_dependency_wait();                                 // the pieces come from the decode grid

    int R = 0;
    const float* lse = partial_lse;
    const float* po = partial_out;
    if (np > 0) {
        if (!own_counts) {
            total = header[0];
            workers = header[1];
            tiles_before = seq_info[2 * s];
            parts_before = seq_info[2 * s + 1];
        }
        const long long first_tile = tiles_before * Hkv + (long long)kvh * tiles;
        const long long first_part = parts_before * Hkv + (long long)kvh * np;
        // worker whose range [floor(T w / W), floor(T (w + 1) / W)) holds tile x: floor(((x + 1) W - 1) / T)
        const long long r0 = first_part + ((first_tile + 1) * workers - 1) / total;
        const long long r1 = first_part + np - 1 + ((first_tile + tiles) * workers - 1) / total;
        R = (int)(r1 - r0 + 1);
        lse += (size_t)r0 * G + hh;                          // stride G
        po += ((size_t)r0 * G + hh) * D + lane * V;          // stride G * D
    }

    // The first kPre rows of this warp's share are requested before the maximum is known: their loads travel
    // together with those of the maximum pass instead of after it (kPre > 0 only for grids of one wave: the
    // registers it takes would cost a many-row grid its occupancy).
    using Vec = typename std::conditional<V == 4, float4, float2>::type;
    float lpre[kPre > 0 ? kPre : 1];
    Vec xpre[kPre > 0 ? kPre : 1];
#pragma unroll
    for (int k = 0; k < kPre; ++k) {
        const int i = sub + k * WPR;
        lpre[k] = -INFINITY;
        if (i < R) {
            lpre[k] = lse[(size_t)i * G];
            xpre[k] = *reinterpret_cast<const Vec*>(po + (size_t)i * G * D);
        }
    }
    float M = -INFINITY;
    for (int i = sub * 32 + lane; i < R; i += WPR * 32) M = fmaxf(M, lse[(size_t)i * G]);
#pragma unroll
    for (int o2 = 16; o2 >= 1; o2 >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o2));
    if (WPR > 1) {
        if (lane == 0) s_max[warp] = M;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < WPR; ++w) M = fmaxf(M, s_max[rib * WPR + w]);
    }

    float num[V];
#pragma unroll
    for (int v = 0; v < V; ++v) num[v] = 0.f;
    float den = 0.f;
    auto add_row = [&](float l, Vec x) {
        if (l > -INFINITY) {                                  // false for the empty numbers: their rows hold nothing
            const float w = ex2((l - M) * kLog2e);
            den += w;
            num[0] = fmaf(w, x.x, num[0]);
            num[1] = fmaf(w, x.y, num[1]);
            if constexpr (V == 4) {
                num[2] = fmaf(w, x.z, num[2]);
                num[3] = fmaf(w, x.w, num[3]);
            }
        }
    };
#pragma unroll
    for (int k = 0; k < kPre; ++k) add_row(lpre[k], xpre[k]);
#pragma unroll 4
    for (int i = sub + kPre * WPR; i < R; i += WPR)
        add_row(lse[(size_t)i * G], *reinterpret_cast<const Vec*>(po + (size_t)i * G * D));
#pragma unroll
    for (int v = 0; v < V; ++v) s_num[warp][lane * V + v] = num[v];
    if (lane == 0) s_den[warp] = den;
    __syncthreads();
    if (!active) return;
    T* o = out + (size_t)row * D;
    for (int d = sub * 32 + lane; d < D; d += WPR * 32) {
        float a = 0.f, b = 0.f;
#pragma unroll
        for (int w = 0; w < WPR; ++w) {
            a += s_num[rib * WPR + w][d];
            b += s_den[rib * WPR + w];
        }
        const float r = np > 0 ? a / b : 0.f;                 // an empty sequence gives a zero row
        if constexpr (sizeof(T) == 2) o[d] = __float2bfloat16_rn(r);
        else o[d] = r;
    }
}

template <typename T, int D>
static int launch_reduce_t(void* out, const float* partial_out, const float* partial_lse,
                           const int32_t* context_lens, int B, int Hq, int partition_size, int max_partitions,
                           int window, cudaStream_t stream) {
    return launch_dependent(reduce_kernel<T, D>, dim3((unsigned)B * (unsigned)Hq), dim3(kReduceWarps * 32), 0, stream,
                            static_cast<T*>(out), partial_out, partial_lse, context_lens, Hq, partition_size,
                            max_partitions, window);
}

int launch_reduce(void* out, const float* partial_out, const float* partial_lse, const int32_t* context_lens,
                  int B, int Hq, int D, int partition_size, int max_partitions, int window, int dtype,
                  cudaStream_t stream) {
    if (dtype == OPT_GQA_BF16) {
        if (D == 128)
            return launch_reduce_t<__nv_bfloat16, 128>(out, partial_out, partial_lse, context_lens, B, Hq,
                                                       partition_size, max_partitions, window, stream);
        return launch_reduce_t<__nv_bfloat16, 64>(out, partial_out, partial_lse, context_lens, B, Hq, partition_size,
                                                  max_partitions, window, stream);
    }
    if (D == 128)
        return launch_reduce_t<float, 128>(out, partial_out, partial_lse, context_lens, B, Hq, partition_size,
                                           max_partitions, window, stream);
    return launch_reduce_t<float, 64>(out, partial_out, partial_lse, context_lens, B, Hq, partition_size,
                                      max_partitions, window, stream);
}

template <typename T, int D, int WPR, int kPre = 0>
static int launch_reduce_balanced_w(void* out, const char* ws, const BalancedLayout& L, const int32_t* context_lens,
                                    int B, int Hq, int Hkv, int partition_size, int window, long long gw,
                                    cudaStream_t stream) {
    const int rows = B * Hq, rpb = kBalWarps / WPR;
    return launch_dependent(reduce_balanced_kernel<T, D, WPR, kPre>, dim3((unsigned)((rows + rpb - 1) / rpb)),
                            dim3(kBalWarps * 32), 0, stream, static_cast<T*>(out),
                            reinterpret_cast<const float*>(ws + L.out), reinterpret_cast<const float*>(ws + L.lse),
                            reinterpret_cast<const long long*>(ws + L.header),
                            reinterpret_cast<const long long*>(ws + L.seq_info), context_lens, rows, Hq, Hkv,
                            partition_size, window, B, gw);
}

template <typename T, int D>
static int launch_reduce_balanced_t(void* out, const char* ws, const BalancedLayout& L, const int32_t* context_lens,
                                    int B, int Hq, int Hkv, int partition_size, int window, long long gw,
                                    cudaStream_t stream) {
    // About 8192 warps in all: 8 per row for a few long rows, 1 per row for batches of many rows.
    const long long rows = (long long)B * Hq;
    if (rows <= 256) return launch_reduce_balanced_w<T, D, 8, 12>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
    if (rows <= 1024) return launch_reduce_balanced_w<T, D, 8, 2>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
    if (rows <= 2048) return launch_reduce_balanced_w<T, D, 4, 2>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
    if (rows <= 4096) return launch_reduce_balanced_w<T, D, 2, 4>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
    // Batches of many rows are mostly short rows (a few pieces each): four preloaded rows cover them in one round trip.
    return launch_reduce_balanced_w<T, D, 1, 4>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
}

int launch_reduce_balanced(void* out, const void* workspace, const int32_t* context_lens, int B, int Hq, int Hkv,
                           int D, int partition_size, int max_partitions, int window, int dtype, cudaStream_t stream) {
    const BalancedLayout L = balanced_layout(B, Hq, Hkv, D, max_partitions);
    const char* ws = static_cast<const char*>(workspace);
    // workers of the decode grid that filled the workspace (0: unknown, the kernel reads the count from the workspace)
    const long long gw = stream_grid_workers(B, Hkv, max_partitions, partition_size);
    if (dtype == OPT_GQA_BF16) {
        if (D == 128)
            return launch_reduce_balanced_t<__nv_bfloat16, 128>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
        return launch_reduce_balanced_t<__nv_bfloat16, 64>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
    }
    if (D == 128) return launch_reduce_balanced_t<float, 128>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
    return launch_reduce_balanced_t<float, 64>(out, ws, L, context_lens, B, Hq, Hkv, partition_size, window, gw, stream);
}

}  // namespace optgqa

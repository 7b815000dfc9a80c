// Paged GQA-ALiBi decode attention for sm_100a (Algorithm 2, "Compute context
// attention with caches"; Eq. 3-5; long-sequence partitioning).
//
// One CTA per (context partition, KV head, sequence).  The CTA streams the K and V
// chunks of its partition through shared memory ONCE for all G query heads of the
// group ("Shared Key-Value").  Work inside the CTA is split by 16-token tiles: warp
// w owns tiles w, w+4, ... and runs its own two-stage ring -- lane 0 enqueues 1-D
// bulk async copies (K tile + V tile, contiguous in the [page, head, slot, dim]
// layout) that complete on the warp's own mbarrier, so no CTA-wide barrier sits in
// the streaming loop.  Per tile a warp computes
//   s[g][j] = <q_g * scale*log2e, k_j> + slope_g*log2e*(j - (n-1))          (Eq. 3)
// with 16 lanes per token row (two rows per step), folds the 16 partial dot
// products of all G heads with a reduce-scatter butterfly, keeps a running
// maximum / denominator per head (online form of Eq. 4) and accumulates
// p[g][j] * v_j in fp32 (Eq. 5).  Warps are merged through shared memory at the end
// and the CTA writes either the final rows or the partition's normalised partial
// result with its log-sum-exp.
#include "common.cuh"

namespace optgqa {

struct DecodeParams {
    void* out;
    const void* q;
    const char* k_cache;
    const char* v_cache;
    const int32_t* block_tables;
    const int32_t* context_lens;
    const float* slopes;
    float* partial_out;
    float* partial_lse;
    int* status;
    float scale;
    int max_blocks;
    int num_blocks;
    int Hq;
    int Hkv;
    int bs;
    int partition_size;
    int max_partitions;
    int window;             // > 0: only the last `window` keys of each sequence are attended to
};

constexpr int kTileTok = 16;   // tokens per tile (one ring stage holds a K tile and a V tile)
constexpr int kWarps = 4;      // warps per CTA, each with a private ring
constexpr int kStages = 2;     // ring depth per warp
constexpr unsigned kFull = 0xffffffffu;

template <typename T, int D, int G>
struct DecodeCfg {
    static constexpr int ES = (int)sizeof(T);
    static constexpr int EPL = D / 16;               // elements of a row owned by one lane
    static constexpr int NC2 = EPL / 2;              // ... as float2
    static constexpr int ROWB = D * ES;              // bytes per token row
    static constexpr int TILE_BYTES = kTileTok * ROWB;
    static constexpr int WARP_RING = kStages * 2 * TILE_BYTES;
    static constexpr int PBUF_FLOATS = kTileTok * G * 2;   // (p,p) pairs of one tile
    static constexpr int OFF_PBUF = kWarps * WARP_RING;
    static constexpr int OFF_ABUF = OFF_PBUF + kWarps * PBUF_FLOATS * 4;
    static constexpr int OFF_M = OFF_ABUF + kWarps * G * 4;
    static constexpr int OFF_L = OFF_M + kWarps * G * 4;
    static constexpr int OFF_BAR = (OFF_L + kWarps * G * 4 + 7) & ~7;
    static constexpr int SMEM = OFF_BAR + kWarps * kStages * 8;
    static constexpr int MIN_CTAS = (220 * 1024 / (SMEM + 1024)) >= 3 ? 3 : ((220 * 1024 / (SMEM + 1024)) >= 2 ? 2 : 1);
    static_assert(G * D * 4 <= WARP_RING, "merge buffer must fit in the warp's ring");
};

// Dimension index of the e-th element a lane owns (c = lane & 15).
template <typename T, int D>
__device__ __forceinline__ int dim_of(int c, int e) {
    constexpr int ROWB = D * (int)sizeof(T);
    if (ROWB <= 256) return c * (D / 16) + e;
    return (e >> 2) * 64 + c * 4 + (e & 3);   // fp32, D = 128: two conflict-free 16-byte vectors per lane
}

// One lane's slice of a token row in shared memory, widened to fp32 pairs.
template <typename T, int D>
__device__ __forceinline__ void load_row(const char* row, int c, float2 (&x)[D / 32]) {
    if constexpr (sizeof(T) == 2 && D == 128) {
        uint4 w = *reinterpret_cast<const uint4*>(row + c * 16);
        x[0] = bf16x2_to_float2(w.x);
        x[1] = bf16x2_to_float2(w.y);
        x[2] = bf16x2_to_float2(w.z);
        x[3] = bf16x2_to_float2(w.w);
    } else if constexpr (sizeof(T) == 2 && D == 64) {
        uint2 w = *reinterpret_cast<const uint2*>(row + c * 8);
        x[0] = bf16x2_to_float2(w.x);
        x[1] = bf16x2_to_float2(w.y);
    } else if constexpr (sizeof(T) == 4 && D == 64) {
        float4 w = *reinterpret_cast<const float4*>(row + c * 16);
        x[0] = make_float2(w.x, w.y);
        x[1] = make_float2(w.z, w.w);
    } else {
        float4 w0 = *reinterpret_cast<const float4*>(row + c * 16);
        float4 w1 = *reinterpret_cast<const float4*>(row + 256 + c * 16);
        x[0] = make_float2(w0.x, w0.y);
        x[1] = make_float2(w0.z, w0.w);
        x[2] = make_float2(w1.x, w1.y);
        x[3] = make_float2(w1.z, w1.w);
    }
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Bit reversal of the low log2(G) bits of the lane id: the head whose score the lane
// ends up holding after the reduce-scatter below.
template <int G>
__device__ __forceinline__ int lane_head(int lane) {
    int h = 0;
#pragma unroll
    for (int b = 0; (1 << b) < G; ++b) h |= ((lane >> b) & 1) * (G >> (b + 1));
    return h;
}

// a[s] holds the lane's partial dot product for head (s ^ lane_head(lane)).  Sums over
// the 16 lanes of a half-warp; returns the total for head lane_head(lane).  Each
// scatter stage keeps the lower half of the slots and receives the partner's upper
// half, which by construction are the same heads, so no selects are needed.
template <int G>
__device__ __forceinline__ float reduce_heads(float (&a)[G]) {
    int mask = 1;
#pragma unroll
    for (int half = G / 2; half >= 1; half /= 2, mask *= 2) {
#pragma unroll
        for (int i = 0; i < half; ++i) a[i] += __shfl_xor_sync(kFull, a[i + half], mask);
    }
#pragma unroll
    for (; mask < 16; mask *= 2) a[0] += __shfl_xor_sync(kFull, a[0], mask);
    return a[0];
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kWarps * 32, DecodeCfg<T, D, G>::MIN_CTAS)
decode_kernel(const DecodeParams p) {
    using C = DecodeCfg<T, D, G>;
    constexpr int NC2 = C::NC2;
    extern __shared__ __align__(128) char smem[];

    grid_dependency_launch();   // the grid after this one (the reduce) may start its own prologue
    const uint64_t read_once = l2_policy_evict_first();     // every K/V byte is read exactly once
    const int part = blockIdx.x, kvh = blockIdx.y, s = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = lane >> 4, c = lane & 15;
    const int n = p.context_lens[s];
    const bool split = p.partition_size > 0;
    const int start = p.window > 0 ? max(0, n - p.window) : 0;     // first attended key (local mask)
    const int t0 = max(split ? part * p.partition_size : 0, start);
    const int t1 = split ? min((part + 1) * p.partition_size, n) : n;

    if (t0 >= t1) {
        // Empty range.  A single-pass call still owes zero rows for an empty sequence.  The wait comes first all the
        // same: an earlier kernel of the stream may still be reading out, and a grid none of whose CTAs waited could
        // finish before its predecessor.
        grid_dependency_wait();
        if (!split) {
            T* o = static_cast<T*>(p.out) + ((size_t)s * p.Hq + (size_t)kvh * G) * D;
            for (int e = threadIdx.x; e < G * D; e += blockDim.x) store_out(o + e, 0.f);
        }
        return;
    }

    char* ring = smem + warp * C::WARP_RING;
    float2* pbuf = reinterpret_cast<float2*>(smem + C::OFF_PBUF) + warp * (C::PBUF_FLOATS / 2);
    float* abuf = reinterpret_cast<float*>(smem + C::OFF_ABUF) + warp * G;
    float* mbuf = reinterpret_cast<float*>(smem + C::OFF_M);
    float* lbuf = reinterpret_cast<float*>(smem + C::OFF_L);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR) + warp * kStages;

    const int tpp = p.bs / kTileTok;                       // tiles per page
    const int first_tile = t0 / kTileTok;
    const int ntiles = (t1 + kTileTok - 1) / kTileTok - first_tile;
    const int cnt = ntiles > warp ? (ntiles - warp + kWarps - 1) / kWarps : 0;   // tiles of this warp
    const int32_t* table = p.block_tables + (size_t)s * p.max_blocks;
    const int hl = lane_head<G>(lane);

    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kStages; ++i) mbar_init(&bars[i], 1);
        fence_barrier_init();
    }
    __syncwarp();

    // Physical pages of this warp's tiles, 32 at a time, one block ahead of the issue index.
    auto load_pages = [&](int kb) -> int {
        int k = kb + lane;
        // Index held inside the table and page id inside the pool: index data that breaks the caller's promises
        // gives a wrong row, not a copy from outside the cache.
        const int page = k < cnt ? __ldg(table + min((first_tile + warp + k * kWarps) / tpp, p.max_blocks - 1)) : 0;
        return min(max(page, 0), p.num_blocks - 1);
    };
    int pages_cur = load_pages(0), pages_next = load_pages(32), blk = 0;

    auto issue = [&](int k) {
        if ((k >> 5) != blk) {
            pages_cur = pages_next;
            ++blk;
            pages_next = load_pages((blk + 1) * 32);
        }
        const int phys = __shfl_sync(kFull, pages_cur, k & 31);
        if (lane == 0) {
            const int tt = first_tile + warp + k * kWarps;
            const size_t off = (((size_t)phys * p.Hkv + kvh) * p.bs + (size_t)(tt % tpp) * kTileTok) * C::ROWB;
            char* dst = ring + (k % kStages) * 2 * C::TILE_BYTES;
            uint64_t* bar = &bars[k % kStages];
            mbar_expect_tx(bar, 2 * C::TILE_BYTES);
            bulk_g2s_hint(dst, p.k_cache + off, C::TILE_BYTES, bar, read_once);
            bulk_g2s_hint(dst + C::TILE_BYTES, p.v_cache + off, C::TILE_BYTES, bar, read_once);
        }
    };

    grid_dependency_wait();     // the cache may still be receiving this step's appended tokens
#pragma unroll
    for (int k = 0; k < kStages; ++k)
        if (k < cnt) issue(k);

    // q of the group, pre-multiplied by scale*log2e; slot g holds head g ^ hl (see reduce_heads).
    float2 q2[G][NC2];
    {
        const T* qg = static_cast<const T*>(p.q) + ((size_t)s * p.Hq + (size_t)kvh * G) * D;
        const float qs = p.scale * kLog2e;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const T* qh = qg + (size_t)(g ^ hl) * D;
#pragma unroll
            for (int e = 0; e < NC2; ++e) {
                q2[g][e].x = to_float(qh[dim_of<T, D>(c, 2 * e)]) * qs;
                q2[g][e].y = to_float(qh[dim_of<T, D>(c, 2 * e + 1)]) * qs;
            }
        }
    }
    const float slope2 = p.slopes ? p.slopes[kvh * G + hl] * kLog2e : 0.f;

    float2 acc[G][NC2];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < NC2; ++e) acc[g][e] = make_float2(0.f, 0.f);
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    int k = 0;

    for (; k < cnt; ++k) {
        const int st = k % kStages;
        const char* kst = ring + st * 2 * C::TILE_BYTES;
        const char* vst = kst + C::TILE_BYTES;
        ok = __all_sync(kFull, mbar_wait(&bars[st], (k / kStages) & 1, p.status));
        if (!ok) break;

        const int j0 = (first_tile + warp + k * kWarps) * kTileTok;    // first token of the tile
        const int valid = min(kTileTok, t1 - j0);
        if (valid < kTileTok) {
            // Rows past the end of the sequence hold whatever the page held: zero the V rows so that
            // 0 * garbage cannot produce NaN (their scores are masked below).
            char* vz = const_cast<char*>(vst);
            for (int r = valid + half; r < kTileTok; r += 2)
                for (int b = c * 16; b < C::ROWB; b += 256) *reinterpret_cast<uint4*>(vz + r * C::ROWB + b) = make_uint4(0, 0, 0, 0);
            __syncwarp();
        }

        // ---- scores of the tile: lane ends with sc[i] = score of token j0 + 2i + half, head hl
        float sc[kTileTok / 2];
#pragma unroll
        for (int i = 0; i < kTileTok / 2; ++i) {
            const int r = 2 * i + half;
            float2 kk[NC2];
            load_row<T, D>(kst + r * C::ROWB, c, kk);
            float a[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float2 t = __fmul2_rn(kk[0], q2[g][0]);
#pragma unroll
                for (int e = 1; e < NC2; ++e) t = __ffma2_rn(kk[e], q2[g][e], t);
                a[g] = t.x + t.y;
            }
            float v = reduce_heads<G>(a);
            const int j = j0 + r;
            v = fmaf(slope2, (float)(j - (n - 1)), v);
            sc[i] = (j < t1 && j >= t0) ? v : -INFINITY;
        }

        // ---- online softmax update (per head, shared by both half-warps)
        float mx = sc[0];
#pragma unroll
        for (int i = 1; i < kTileTok / 2; ++i) mx = fmaxf(mx, sc[i]);
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 16));
        const float m_new = fmaxf(m, mx);
        const float alpha = ex2(m - m_new);
        const bool rescale = __any_sync(kFull, m_new > m);
        m = m_new;
        float psum = 0.f;
#pragma unroll
        for (int i = 0; i < kTileTok / 2; ++i) {
            const float pj = ex2(sc[i] - m_new);
            psum += pj;
            pbuf[(2 * i + half) * G + hl] = make_float2(pj, pj);
        }
        l = fmaf(l, alpha, psum);
        if (rescale) abuf[hl] = alpha;
        __syncwarp();
        if (rescale) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float a = abuf[g];
                const float2 a2 = make_float2(a, a);
#pragma unroll
                for (int e = 0; e < NC2; ++e) acc[g][e] = __fmul2_rn(acc[g][e], a2);
            }
        }

        // ---- weighted sum of V: each half-warp adds its own token rows
#pragma unroll
        for (int i = 0; i < kTileTok / 2; ++i) {
            const int r = 2 * i + half;
            float2 vv[NC2];
            load_row<T, D>(vst + r * C::ROWB, c, vv);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float2 pp = pbuf[r * G + g];
#pragma unroll
                for (int e = 0; e < NC2; ++e) acc[g][e] = __ffma2_rn(vv[e], pp, acc[g][e]);
            }
        }

        __syncwarp();
        if (k + kStages < cnt) {
            fence_proxy_async();
            issue(k + kStages);
        }
    }

    if (!ok) {
        // A wait gave up (already recorded).  Give the copies still in flight one more bounded
        // chance to land before this CTA's shared memory is released.
        for (int kk = k; kk < min(cnt, k + kStages); ++kk) mbar_wait(&bars[kk % kStages], (kk / kStages) & 1, p.status);
    }

    // ---- fold the two half-warps, then park (m, l, acc) in this warp's ring for the CTA-wide merge
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int e = 0; e < NC2; ++e) {
            acc[g][e].x += __shfl_xor_sync(kFull, acc[g][e].x, 16);
            acc[g][e].y += __shfl_xor_sync(kFull, acc[g][e].y, 16);
        }
    l += __shfl_xor_sync(kFull, l, 16);
    float* macc = reinterpret_cast<float*>(ring);
    if (half == 0) {
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < NC2; ++e)
                *reinterpret_cast<float2*>(macc + g * D + dim_of<T, D>(c, 2 * e)) = acc[g][e];
    }
    mbuf[warp * G + hl] = m;
    lbuf[warp * G + hl] = l;
    __syncthreads();

    const int nw = min(kWarps, ntiles);   // warps that saw at least one tile
    for (int e = threadIdx.x; e < G * D; e += blockDim.x) {
        const int g = e / D, d = e % D;
        float M = mbuf[g];
        for (int w = 1; w < nw; ++w) M = fmaxf(M, mbuf[w * G + g]);
        float num = 0.f, den = 0.f;
        for (int w = 0; w < nw; ++w) {
            const float f = ex2(mbuf[w * G + g] - M);
            den = fmaf(f, lbuf[w * G + g], den);
            num = fmaf(f, reinterpret_cast<const float*>(smem + w * C::WARP_RING)[e], num);
        }
        const float o = num / den;
        const size_t row = (size_t)s * p.Hq + (size_t)kvh * G + g;
        if (split) {
            p.partial_out[(row * p.max_partitions + part) * D + d] = o;
            if (d == 0) p.partial_lse[row * p.max_partitions + part] = (M + log2f(den)) * kLn2;
        } else {
            store_out(static_cast<T*>(p.out) + row * D + d, o);
        }
    }
}

template <typename T, int D, int G>
static int launch_one(const DecodeParams& p, int B, cudaStream_t stream) {
    using C = DecodeCfg<T, D, G>;
    static std::atomic<bool> configured[kMaxDevices];
    if (!ensure_smem_limit(decode_kernel<T, D, G>, C::SMEM, configured)) return OPT_GQA_ERR_CUDA;
    dim3 grid(p.partition_size > 0 ? p.max_partitions : 1, p.Hkv, B);
    return launch_dependent(decode_kernel<T, D, G>, grid, dim3(kWarps * 32), C::SMEM, stream, p);
}

template <typename T, int D>
static int launch_g(const DecodeParams& p, int B, int G, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_one<T, D, 1>(p, B, stream);
        case 2: return launch_one<T, D, 2>(p, B, stream);
        case 4: return launch_one<T, D, 4>(p, B, stream);
        case 8: return launch_one<T, D, 8>(p, B, stream);
    }
    return OPT_GQA_ERR_SHAPE;
}

int launch_decode(void* out, const void* q, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                  int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes, float scale,
                  int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size, float* partial_out,
                  float* partial_lse, int max_partitions, int window, int dtype, int* device_status,
                  cudaStream_t stream) {
    if (num_blocks <= 0 || num_blocks > 0x7fffffffll) return OPT_GQA_ERR_SHAPE;
    DecodeParams p;
    p.num_blocks = (int)num_blocks;
    p.out = out;
    p.q = q;
    p.k_cache = static_cast<const char*>(k_cache);
    p.v_cache = static_cast<const char*>(v_cache);
    p.block_tables = block_tables;
    p.context_lens = context_lens;
    p.slopes = alibi_slopes;
    p.partial_out = partial_out;
    p.partial_lse = partial_lse;
    p.status = device_status;
    p.scale = scale;
    p.max_blocks = max_blocks_per_seq;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.bs = bs;
    p.partition_size = partition_size;
    p.max_partitions = max_partitions;
    p.window = window;
    const int G = Hq / Hkv;
    if (dtype == OPT_GQA_BF16) {
        if (D == 128) return launch_g<__nv_bfloat16, 128>(p, B, G, stream);
        if (D == 64) return launch_g<__nv_bfloat16, 64>(p, B, G, stream);
    } else {
        if (D == 128) return launch_g<float, 128>(p, B, G, stream);
        if (D == 64) return launch_g<float, 64>(p, B, G, stream);
    }
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace optgqa

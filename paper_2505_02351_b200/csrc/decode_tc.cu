// Paged GQA-ALiBi decode attention for bf16 caches on sm_100a, group-as-tile form
// (Algorithm 2, "Compute context attention with caches"; Eq. 3-5; long-sequence
// partitioning).
//
// Same decomposition as the SIMT kernel in decode.cu -- one CTA per (context
// partition, KV head, sequence), every K/V tile brought on-chip once for the whole
// query group, one private two-stage ring per warp -- but the G query heads of the
// group are the rows of an m16n8k16 tile, so that Eq. 3's dot products and Eq. 5's
// weighted sum run on the tensor pipe and the ALUs only see the softmax.  With G = 8
// the arithmetic intensity is 8 flop per cache byte, which the fp32 FMA pipe cannot
// sustain at HBM speed (measured: 40 % of the copy bandwidth at 46 % issue-slot use).
//
// Tiles are fetched by 2-D TMA with the 128-byte swizzle, which makes both the
// row-wise ldmatrix of K (B operand of q k^T) and the transposing ldmatrix of V
// (B operand of p V) bank-conflict free.  Scores stay in fp32 registers; p is
// rounded to bf16 only as the tensor-core operand and the denominator sums the same
// rounded values; accumulation is fp32.
#include "tma_mma.cuh"

namespace optgqa {

namespace {

// Warps per CTA (each with a private ring) and CTAs per SM the register budget is held to, for the two uses of the
// kernel.  One CTA per (sequence, KV head) has the whole context to itself: twelve warps, one CTA per SM (192 KiB of
// rings; measured on 256 streams of 512-2048 tokens: 8 warps 31.6 us, 10 30.7, 12 28.9, 13 32.2 and 14 31.4 -- past
// twelve the register cap of 128 spills and the warps no longer divide over the four schedulers --, 6 warps x 2 CTAs
// 32.5, 4 x 3 35.3; on 2048 ragged streams 218.7 with 8 warps, 204.8 with 12).  One CTA per (sequence, KV head,
// partition) has a few hundred tokens: two warps, six CTAs per SM, so that the CTA scheduler has many small items to
// even out (one partial per 512-token partition on long contexts: 1 warp x 12 CTAs 69.2 us, 2 x 6 68.7, 2 x 5 69.3,
// 3 x 4 73.4, 4 x 3 75.7).
constexpr int kWarpsSingle = 12, kCtasSingle = 1;
constexpr int kWarpsSplit = 2, kCtasSplit = 6;
constexpr int kTileTok = 16;                 // tokens per tile (one ring stage holds a K tile and a V tile)
constexpr int kStages = 2;                   // ring depth per warp
constexpr unsigned kFull = 0xffffffffu;

struct TcParams {
    void* out;
    const __nv_bfloat16* q;
    const int32_t* block_tables;
    const int32_t* context_lens;
    const float* slopes;
    float* partial_out;
    float* partial_lse;
    int* status;
    float scale;
    int max_blocks;
    int Hq;
    int Hkv;
    int bs;
    int partition_size;
    int max_partitions;
    int B;
    // fused store of the step's new tokens (all null when the cache already holds them)
    const uint4* k_new;
    const uint4* v_new;
    uint4* k_cache_w;
    uint4* v_cache_w;
    const int64_t* slot_mapping;
};

template <int D, int G, int kWarps>
struct TcCfg {
    static constexpr int NBOX = D / 64;                   // 128-byte-wide boxes per token row
    static constexpr int BOX_BYTES = kTileTok * 128;      // 16 rows x 128 B
    static constexpr int TILE_BYTES = NBOX * BOX_BYTES;   // K (or V) bytes per tile
    static constexpr int WARP_RING = kStages * 2 * TILE_BYTES;
    static constexpr int OFF_M = kWarps * WARP_RING;
    static constexpr int OFF_L = OFF_M + kWarps * G * 4;
    static constexpr int OFF_BAR = (OFF_L + kWarps * G * 4 + 7) & ~7;
    static constexpr int SMEM = OFF_BAR + kWarps * kStages * 8 + 1024;   // + slack to align the ring to 1 KB
    static_assert(G * D * 4 <= WARP_RING, "merge buffer must fit in the warp's ring");
};

// d += a * b, m16n8k16, bf16 operands, fp32 accumulate.  Rows 8..15 of a are zero here (a1 = a3 = 0).
__device__ __forceinline__ void mma_bf16_rows8(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of token row `row` inside a tile stored as
// NBOX boxes of 16 rows x 128 B with the 128-byte swizzle (chunk index XOR row mod 8).
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * (kTileTok * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int D, int G, int kWarps, int kMinCtas>
__global__ void __launch_bounds__(kWarps * 32, kMinCtas)
decode_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const TcParams p) {
    using C = TcCfg<D, G, kWarps>;
    constexpr int KS = D / 16;    // k-steps of q k^T
    constexpr int NT = D / 8;     // n-tiles of p V
    extern __shared__ char smem_raw[];
    char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);

    grid_dependency_launch();   // the grid after this one (the reduce) may start its own prologue
    const uint64_t read_once = l2_policy_evict_first();     // every K/V byte is read exactly once
    const uint64_t keep = l2_policy_evict_last();           // the partial results are read by the merge that follows
    // Work item of this CTA.  The KV head runs fastest: CTAs that start together read the same pages (a page holds the
    // rows of all KV heads side by side), which keeps the DRAM accesses of a moment close together.  The partition
    // index runs slowest, so that the grid ends with the high partition numbers, which only the longest sequences
    // have: the last CTAs to start are few and short.
    const int kvh = blockIdx.x % p.Hkv, s = (blockIdx.x / p.Hkv) % p.B, part = blockIdx.x / (p.B * p.Hkv);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;      // fragment row (query head of the group) and column pair
    const bool split = p.partition_size > 0;
    const int t0 = split ? part * p.partition_size : 0;
    const int tpp = p.bs / kTileTok;
    const int first_tile = t0 / kTileTok;
    const int32_t* table = p.block_tables + (size_t)s * p.max_blocks;
    // Page ids of this warp's tiles, 32 at a time.  The index is held inside the table, so the loads do not depend on
    // the sequence's length (they travel together with the load of n instead of after it; ids past the end are never
    // used) and a length beyond max_blocks * bs gives a wrong row, not a stray access.
    auto load_pages = [&](int kb) -> int {
        return __ldg(table + min((first_tile + warp + (kb + lane) * kWarps) / tpp, p.max_blocks - 1));
    };
    int pages_cur = load_pages(0), pages_next = load_pages(32), blk = 0;
    const int n = p.context_lens[s];
    const int t1 = split ? min(t0 + p.partition_size, n) : n;

    if (t0 >= t1) {
        // Empty range.  The wait comes first all the same: an earlier kernel of the stream may still be reading out,
        // and a grid none of whose CTAs waited could finish before its predecessor.
        grid_dependency_wait();
        if (!split) {
            __nv_bfloat16* o = static_cast<__nv_bfloat16*>(p.out) + ((size_t)s * p.Hq + (size_t)kvh * G) * D;
            for (int e = threadIdx.x; e < G * D; e += blockDim.x) o[e] = __float2bfloat16_rn(0.f);
        }
        return;
    }

    char* ring = smem + warp * C::WARP_RING;
    float* mbuf = reinterpret_cast<float*>(smem + C::OFF_M);
    float* lbuf = reinterpret_cast<float*>(smem + C::OFF_L);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR) + warp * kStages;

    const int ntiles = (t1 + kTileTok - 1) / kTileTok - first_tile;
    const int cnt = ntiles > warp ? (ntiles - warp + kWarps - 1) / kWarps : 0;

    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kStages; ++i) mbar_init(&bars[i], 1);
        fence_barrier_init();
    }
    __syncwarp();

    auto issue = [&](int k) {
        if ((k >> 5) != blk) {
            pages_cur = pages_next;
            ++blk;
            pages_next = load_pages((blk + 1) * 32);
        }
        const int phys = __shfl_sync(kFull, pages_cur, k & 31);
        if (p.k_new && first_tile + warp + k * kWarps == (n - 1) / kTileTok) {
            // The step's new token of this sequence lies in the tile about to be fetched (Algorithm 2, "Store reshaped
            // K, V into C_K, C_V"): store its K and V rows of this head first, as the slot-mapped write would, and order
            // the stores before the bulk copy.  The tile belongs to this warp alone, so nobody reads the row earlier.
            const long long slot = __ldg(p.slot_mapping + s);
            if (slot >= 0) {
                constexpr int VEC = D * 2 / 16;                  // 16-byte vectors per row
                if (lane < 2 * VEC) {
                    const bool is_v = lane >= VEC;
                    const int vi = lane % VEC;
                    const size_t src = ((size_t)s * p.Hkv + kvh) * VEC + vi;
                    const size_t dst = (((size_t)(slot / p.bs) * p.Hkv + kvh) * p.bs + (size_t)(slot % p.bs)) * VEC + vi;
                    if (is_v) p.v_cache_w[dst] = __ldg(p.v_new + src);
                    else p.k_cache_w[dst] = __ldg(p.k_new + src);
                }
                asm volatile("fence.proxy.async.global;" ::: "memory");
            }
            __syncwarp();
        }
        if (lane == 0) {
            const int tt = first_tile + warp + k * kWarps;
            const int row = (phys * p.Hkv + kvh) * p.bs + (tt % tpp) * kTileTok;   // row of the [rows, D] view
            char* dst = ring + (k % kStages) * 2 * C::TILE_BYTES;
            uint64_t* bar = &bars[k % kStages];
            mbar_expect_tx(bar, 2 * C::TILE_BYTES);
#pragma unroll
            for (int b = 0; b < C::NBOX; ++b) {
                tma_load_2d_hint(dst + b * C::BOX_BYTES, &map_k, b * 64, row, bar, read_once);
                tma_load_2d_hint(dst + C::TILE_BYTES + b * C::BOX_BYTES, &map_v, b * 64, row, bar, read_once);
            }
        }
    };

    grid_dependency_wait();     // the cache may still be receiving this step's appended tokens
#pragma unroll
    for (int k = 0; k < kStages; ++k)
        if (k < cnt) issue(k);

    // A fragments of q (rows = heads of the group; rows >= G are zero): a0 = dims 16s+2t,+1; a2 = dims 16s+8+2t,+1.
    uint32_t qa[KS][2];
    {
        const uint32_t* qh =
            reinterpret_cast<const uint32_t*>(p.q + ((size_t)s * p.Hq + (size_t)kvh * G + (g < G ? g : 0)) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = g < G ? qh[ks * 8 + t] : 0u;
            qa[ks][1] = g < G ? qh[ks * 8 + 4 + t] : 0u;
        }
    }
    const float qscale = p.scale * kLog2e;
    const float slope2 = (p.slopes && g < G) ? p.slopes[kvh * G + g] * kLog2e : 0.f;

    float o[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    int k = 0;

    // ldmatrix lane roles: lane supplies the address of row (lane & 7) of matrix (lane >> 3).
    const int lrow = lane & 7, lmat = lane >> 3;

    for (; k < cnt; ++k) {
        const int st = k % kStages;
        char* kst = ring + st * 2 * C::TILE_BYTES;
        char* vst = kst + C::TILE_BYTES;
        ok = __all_sync(kFull, mbar_wait(&bars[st], (k / kStages) & 1, p.status));
        if (!ok) break;

        const int j0 = (first_tile + warp + k * kWarps) * kTileTok;
        const int valid = min(kTileTok, t1 - j0);
        if (valid < kTileTok) {
            // zero the V rows past the end of the sequence (whole rows, so the swizzle does not matter)
            for (int r = valid + (lane >> 3); r < kTileTok; r += 4)
#pragma unroll
                for (int b = 0; b < C::NBOX; ++b)
                    *reinterpret_cast<uint4*>(vst + b * C::BOX_BYTES + r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
            __syncwarp();
        }

        // ---- scores: S[head][token] for tokens j0 .. j0+15 as two n-tiles of 8
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const uint32_t kbase = smem_u32(kst);
            const int krow = lrow + 8 * (lmat >> 1);          // matrices 0,1: tokens 0-7; 2,3: tokens 8-15
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t b[4];
                ldmatrix_x4(b, kbase + swz(krow, 2 * ks + (lmat & 1)));
                mma_bf16_rows8(sa, qa[ks][0], qa[ks][1], b[0], b[1]);
                mma_bf16_rows8(sb, qa[ks][0], qa[ks][1], b[2], b[3]);
            }
        }
        // thread holds head g, tokens j0 + {2t, 2t+1} (sa[0], sa[1]) and j0 + 8 + {2t, 2t+1} (sb[0], sb[1])
        float sc[4];
        {
            const int ja = j0 + 2 * t, jb = ja + 8;
            const float rel = (float)(ja - (n - 1));
            sc[0] = fmaf(sa[0], qscale, slope2 * rel);
            sc[1] = fmaf(sa[1], qscale, slope2 * (rel + 1.f));
            sc[2] = fmaf(sb[0], qscale, slope2 * (rel + 8.f));
            sc[3] = fmaf(sb[1], qscale, slope2 * (rel + 9.f));
            sc[0] = ja < t1 ? sc[0] : -INFINITY;
            sc[1] = ja + 1 < t1 ? sc[1] : -INFINITY;
            sc[2] = jb < t1 ? sc[2] : -INFINITY;
            sc[3] = jb + 1 < t1 ? sc[3] : -INFINITY;
        }
        float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
        const float m_new = fmaxf(m, mx);
        const float alpha = ex2(m - m_new);
        const bool rescale = __any_sync(kFull, m_new > m);
        m = m_new;
        // p rounded to bf16 once: the same values feed the tensor core and the denominator
        const __nv_bfloat162 p01 = __floats2bfloat162_rn(ex2(sc[0] - m_new), ex2(sc[1] - m_new));
        const __nv_bfloat162 p23 = __floats2bfloat162_rn(ex2(sc[2] - m_new), ex2(sc[3] - m_new));
        const float2 f01 = __bfloat1622float2(p01), f23 = __bfloat1622float2(p23);
        l = fmaf(l, alpha, (f01.x + f01.y) + (f23.x + f23.y));
        const uint32_t pa0 = *reinterpret_cast<const uint32_t*>(&p01);
        const uint32_t pa2 = *reinterpret_cast<const uint32_t*>(&p23);
        if (rescale) {
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                o[i][0] *= alpha;
                o[i][1] *= alpha;
            }
        }

        // ---- O[head][dim] += P[head][token] * V[token][dim]; V transposed on the fly by ldmatrix.trans
        {
            const uint32_t vbase = smem_u32(vst);
            const int vrow = lrow + 8 * (lmat & 1);           // matrices 0,2: tokens 0-7; 1,3: tokens 8-15
#pragma unroll
            for (int jj = 0; jj < NT / 2; ++jj) {
                uint32_t b[4];
                ldmatrix_x4_trans(b, vbase + swz(vrow, 2 * jj + (lmat >> 1)));
                mma_bf16_rows8(o[2 * jj], pa0, pa2, b[0], b[1]);
                mma_bf16_rows8(o[2 * jj + 1], pa0, pa2, b[2], b[3]);
            }
        }

        __syncwarp();
        if (k + kStages < cnt) {
            fence_proxy_async();
            issue(k + kStages);
        }
    }

    if (!ok) {
        for (int kk = k; kk < min(cnt, k + kStages); ++kk) mbar_wait(&bars[kk % kStages], (kk / kStages) & 1, p.status);
    }

    // ---- per-head denominator over the quad, then park (m, l, O) in this warp's ring for the CTA-wide merge
    l += __shfl_xor_sync(kFull, l, 1);
    l += __shfl_xor_sync(kFull, l, 2);
    float* macc = reinterpret_cast<float*>(ring);
    if (g < G) {
#pragma unroll
        for (int i = 0; i < NT; ++i) *reinterpret_cast<float2*>(macc + g * D + i * 8 + 2 * t) = make_float2(o[i][0], o[i][1]);
        if (t == 0) {
            mbuf[warp * G + g] = m;
            lbuf[warp * G + g] = l;
        }
    }
    __syncthreads();

    const int nw = min(kWarps, ntiles);
    for (int e = threadIdx.x; e < G * D; e += blockDim.x) {
        const int hg = e / D, d = e % D;
        float M = mbuf[hg];
        for (int w = 1; w < nw; ++w) M = fmaxf(M, mbuf[w * G + hg]);
        float num = 0.f, den = 0.f;
        for (int w = 0; w < nw; ++w) {
            const float f = ex2(mbuf[w * G + hg] - M);
            den = fmaf(f, lbuf[w * G + hg], den);
            num = fmaf(f, reinterpret_cast<const float*>(smem + w * C::WARP_RING)[e], num);
        }
        const float r = num / den;
        const size_t row = (size_t)s * p.Hq + (size_t)kvh * G + hg;
        if (split) {
            st_global_hint(p.partial_out + (row * p.max_partitions + part) * D + d, r, keep);
            if (d == 0) st_global_hint(p.partial_lse + row * p.max_partitions + part, (M + log2f(den)) * kLn2, keep);
        } else {
            static_cast<__nv_bfloat16*>(p.out)[row * D + d] = __float2bfloat16_rn(r);
        }
    }
}

template <int D, int G, int kWarps, int kMinCtas>
int launch_shape(const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& p, int B, cudaStream_t stream) {
    using C = TcCfg<D, G, kWarps>;
    static std::atomic<bool> configured[kMaxDevices];
    if (!ensure_smem_limit(decode_tc_kernel<D, G, kWarps, kMinCtas>, C::SMEM, configured)) return OPT_GQA_ERR_CUDA;
    const long long ctas = (long long)(p.partition_size > 0 ? p.max_partitions : 1) * p.Hkv * B;
    if (ctas > 0x7fffffffll) return OPT_GQA_ERR_SHAPE;
    dim3 grid((unsigned)ctas);
    return launch_dependent(decode_tc_kernel<D, G, kWarps, kMinCtas>, grid, dim3(kWarps * 32), C::SMEM, stream, mk, mv,
                            p);
}

template <int D, int G>
int launch_one(const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& p, int B, cudaStream_t stream) {
    if (p.partition_size > 0) return launch_shape<D, G, kWarpsSplit, kCtasSplit>(mk, mv, p, B, stream);
    return launch_shape<D, G, kWarpsSingle, kCtasSingle>(mk, mv, p, B, stream);
}

template <int D>
int launch_g(const CUtensorMap& mk, const CUtensorMap& mv, const TcParams& p, int B, int G, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_one<D, 1>(mk, mv, p, B, stream);
        case 2: return launch_one<D, 2>(mk, mv, p, B, stream);
        case 4: return launch_one<D, 4>(mk, mv, p, B, stream);
        case 8: return launch_one<D, 8>(mk, mv, p, B, stream);
    }
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace

int launch_decode_tc(void* out, const void* q, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                     int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes, float scale,
                     int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                     float* partial_out, float* partial_lse, int max_partitions, int* device_status,
                     cudaStream_t stream, const FusedAppend* append) {
    const uint64_t rows = (uint64_t)num_blocks * (uint64_t)Hkv * (uint64_t)bs;
    if (rows == 0 || rows > 0x7fffffffull) return OPT_GQA_ERR_SHAPE;
    CUtensorMap mk, mv;
    if (!make_cache_map(&mk, k_cache, rows, D, kTileTok) || !make_cache_map(&mv, v_cache, rows, D, kTileTok))
        return OPT_GQA_ERR_CUDA;
    TcParams p;
    p.out = out;
    p.q = static_cast<const __nv_bfloat16*>(q);
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
    p.B = B;
    p.k_new = append ? static_cast<const uint4*>(append->k_new) : nullptr;
    p.v_new = append ? static_cast<const uint4*>(append->v_new) : nullptr;
    p.k_cache_w = append ? static_cast<uint4*>(append->k_cache) : nullptr;
    p.v_cache_w = append ? static_cast<uint4*>(append->v_cache) : nullptr;
    p.slot_mapping = append ? append->slot_mapping : nullptr;
    const int G = Hq / Hkv;
    if (D == 128) return launch_g<128>(mk, mv, p, B, G, stream);
    if (D == 64) return launch_g<64>(mk, mv, p, B, G, stream);
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace optgqa

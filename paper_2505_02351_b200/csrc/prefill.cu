// Multi-token (chunked-prefill) GQA-ALiBi attention over the paged cache on tensor cores,
// warp-level mma form (the prompt branch of Algorithms 1 and 2 with "Create ALiBi bias"
// and the causal mask; Eq. 3-5).  bf16 only.
//
// One CTA per (query block, KV head, sequence).  The G query heads of the group times
// TQ = 128 / G consecutive new tokens form the 128 rows of the CTA's score tile, so a
// K/V tile is brought on-chip once for the whole group ("Shared Key-Value") and every
// tensor-core instruction works on a full 16-row tile.  Eight consumer warps own 16 rows
// each (one head, 16 consecutive tokens); a ninth warp is the producer: it walks the
// block table and fetches 64-token K and V tiles (one 2-D TMA box of 16 token rows x 128
// bytes per page slice, 128-byte swizzle) into a three-stage ring guarded by full/empty
// mbarriers.  Per tile a consumer warp computes S = q k^T (m16n8k16, fp32 accumulate),
// adds the ALiBi term slope_h*(j - pos) and masks j > pos from the indices (Eq. 3; no
// mask or bias matrix exists in memory), keeps the running maximum and denominator of
// Eq. 4 per row, rounds p to bf16 once (the same rounded values feed the tensor core and
// the denominator) and accumulates p V in fp32 (Eq. 5).
#include "tma_mma.cuh"

namespace optgqa {

namespace {

constexpr int kRows = 128;        // rows of the CTA's score tile (G heads x TQ tokens)
constexpr int kConsumers = 8;     // consumer warps, 16 rows each
constexpr int kTK = 64;           // keys per tile
constexpr int kSub = 16;          // token rows per TMA box (one page, or half of a 32-token page)
constexpr int kPStages = 3;
constexpr unsigned kFull = 0xffffffffu;

struct PrefillParams {
    __nv_bfloat16* out;
    const __nv_bfloat16* q;
    const int32_t* q_start_loc;
    const int32_t* block_tables;
    const int32_t* context_lens;
    const float* slopes;
    int* status;
    float scale;
    int max_blocks;
    int Hq;
    int Hkv;
    int bs;
};

template <int D>
struct PrefillCfg {
    static constexpr int NBOX = D / 64;                    // 128-byte-wide column boxes per row
    static constexpr int BOX_BYTES = kTK * 128;            // one column box of a 64-token tile
    static constexpr int TILE_BYTES = NBOX * BOX_BYTES;    // K (or V) bytes per tile
    static constexpr int SUB_BYTES = kSub * 128;           // one TMA box
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    static constexpr int OFF_BAR = kPStages * STAGE_BYTES;
    static constexpr int SMEM = OFF_BAR + 2 * kPStages * 8 + 1024;   // + slack to align the ring to 1 KB
};

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of token row `row` (0 .. 63) inside a tile stored
// as NBOX column boxes of 64 rows x 128 B with the 128-byte swizzle (chunk index XOR row mod 8).
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * (kTK * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi, float& sum) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    const float2 f = __bfloat1622float2(v);
    sum += f.x + f.y;
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <int D, int G>
__global__ void __launch_bounds__((kConsumers + 1) * 32, 1)
prefill_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
               const PrefillParams p) {
    using C = PrefillCfg<D>;
    constexpr int TQ = kRows / G;     // new tokens per query block
    constexpr int KS = D / 16;        // k-steps of q k^T
    constexpr int NT = D / 8;         // n-tiles of p V
    extern __shared__ char smem_raw[];
    char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
    uint64_t* empty = full + kPStages;

    const int kvh = blockIdx.y, s = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qstart = p.q_start_loc[s];
    const int qlen = p.q_start_loc[s + 1] - qstart;
    const int nblk = (qlen + TQ - 1) / TQ;
    if ((int)blockIdx.x >= nblk) {
        grid_dependency_wait();     // a grid none of whose CTAs waited could finish before its predecessor
        return;
    }
    const int qb = nblk - 1 - (int)blockIdx.x;             // the longest-running blocks start first
    const int n = p.context_lens[s];
    const int i_last = min(qlen, (qb + 1) * TQ) - 1;        // last valid new token of this block
    const int pos_last = n - qlen + i_last;                 // its position; the block sees keys 0 .. pos_last
    const int ntiles = pos_last / kTK + 1;

    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < kPStages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], kConsumers);
        }
        fence_barrier_init();
    }
    __syncthreads();
    grid_dependency_wait();     // the cache may still be receiving this step's appended tokens

    if (warp == kConsumers) {
        // ------------------------------------------------------------------ producer warp
        const int32_t* table = p.block_tables + (size_t)s * p.max_blocks;
        const int sub = lane & 3;                           // lanes 0-3 fetch one 16-token slice each
        auto page_of = [&](int kt) -> int {
            const int j = kt * kTK + sub * kSub;
            return (lane < 4 && j < n) ? __ldg(table + j / p.bs) : -1;
        };
        int page = page_of(0);
        bool ok = true;
        int kt = 0;
        for (; kt < ntiles; ++kt) {
            const int st = kt % kPStages;
            const int page_next = kt + 1 < ntiles ? page_of(kt + 1) : -1;
            if (kt >= kPStages) {
                ok = mbar_wait(&empty[st], ((kt / kPStages) - 1) & 1, p.status);
                ok = __all_sync(kFull, ok);
                if (!ok) break;
            }
            const int j0 = kt * kTK;
            const int nsub = min(kTK / kSub, (n - j0 + kSub - 1) / kSub);   // slices that hold cached tokens
            if (lane == 0) mbar_expect_tx(&full[st], (uint32_t)nsub * 2u * C::NBOX * C::SUB_BYTES);
            __syncwarp();
            if (lane < nsub) {
                const int j = j0 + sub * kSub;
                const int row = (page * p.Hkv + kvh) * p.bs + j % p.bs;       // row of the [rows, D] view
                char* kdst = smem + st * C::STAGE_BYTES + sub * C::SUB_BYTES;
                char* vdst = kdst + C::TILE_BYTES;
#pragma unroll
                for (int b = 0; b < C::NBOX; ++b) {
                    tma_load_2d(kdst + b * C::BOX_BYTES, &map_k, b * 64, row, &full[st]);
                    tma_load_2d(vdst + b * C::BOX_BYTES, &map_v, b * 64, row, &full[st]);
                }
            }
            page = page_next;
        }
        // Copies already issued complete whatever the consumers do; before this warp lets go of the CTA's
        // shared memory on the failure path, give them a bounded chance to land.
        if (!ok && lane == 0)
            for (int kk = max(0, kt - kPStages); kk < kt; ++kk)
                mbar_wait(&full[kk % kPStages], (kk / kPStages) & 1, p.status);
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    const int g = lane >> 2, t = lane & 3;
    const int r0 = warp * 16;                     // first row of this warp in the CTA tile
    const int hg = r0 / TQ;                       // head of the group (the same for the warp's 16 rows)
    const int tok0 = r0 % TQ;                     // first token of the warp inside the query block
    const int iA = qb * TQ + tok0 + g, iB = iA + 8;             // new-token indices of rows g and g + 8
    const bool validA = iA < qlen, validB = iB < qlen;
    // Rows past the end of the block are computed as copies of the last valid position and never stored.
    const int posA = n - qlen + min(iA, i_last), posB = n - qlen + min(iB, i_last);
    const int pos_lo = n - qlen + min(qb * TQ + tok0, i_last);          // smallest position in the warp
    const int pos_hi = n - qlen + min(qb * TQ + tok0 + 15, i_last);     // largest
    const int h = kvh * G + hg;

    uint32_t qa[KS][4];
    {
        const uint32_t* qA = reinterpret_cast<const uint32_t*>(p.q + ((size_t)(qstart + min(iA, i_last)) * p.Hq + h) * D);
        const uint32_t* qB = reinterpret_cast<const uint32_t*>(p.q + ((size_t)(qstart + min(iB, i_last)) * p.Hq + h) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qa[ks][0] = __ldg(qA + ks * 8 + t);
            qa[ks][1] = __ldg(qB + ks * 8 + t);
            qa[ks][2] = __ldg(qA + ks * 8 + 4 + t);
            qa[ks][3] = __ldg(qB + ks * 8 + 4 + t);
        }
    }
    const float qscale = p.scale * kLog2e;
    const float slope2 = p.slopes ? p.slopes[h] * kLog2e : 0.f;

    float o[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
    const int lrow = lane & 7, lmat = lane >> 3;
    bool ok = true;

    for (int kt = 0; kt < ntiles; ++kt) {
        const int st = kt % kPStages;
        char* kst = smem + st * C::STAGE_BYTES;
        char* vst = kst + C::TILE_BYTES;
        ok = __all_sync(kFull, mbar_wait(&full[st], (kt / kPStages) & 1, p.status));
        if (!ok) break;
        const int j0 = kt * kTK;

        if (j0 <= pos_hi) {     // otherwise every key of the tile lies after every row of this warp
            if (j0 + kTK > n) {
                // Rows past the end of the sequence hold whatever the page held (or stale shared memory where
                // no page exists): zero the V rows so that 0 * garbage cannot produce NaN.  Every warp clears
                // the same rows with the same value, so the warps need no barrier between them.
                for (int r = (n - j0) + (lane >> 3); r < kTK; r += 4)
#pragma unroll
                    for (int b = 0; b < C::NBOX; ++b)
                        *reinterpret_cast<uint4*>(vst + b * C::BOX_BYTES + r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
                fence_proxy_async();
                __syncwarp();
            }

            // ---- S[row][key] for the tile's 64 keys as eight n-tiles of 8
            float sc[kTK / 8][4];
#pragma unroll
            for (int i = 0; i < kTK / 8; ++i) sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
            {
                const uint32_t kbase = smem_u32(kst);
                const int krow = lrow + 8 * (lmat >> 1);
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
                    for (int nn = 0; nn < kTK / 16; ++nn) {
                        uint32_t b[4];
                        ldmatrix_x4(b, kbase + swz(16 * nn + krow, 2 * ks + (lmat & 1)));
                        mma_bf16(sc[2 * nn], qa[ks], b[0], b[1]);
                        mma_bf16(sc[2 * nn + 1], qa[ks], b[2], b[3]);
                    }
                }
            }
            // thread holds rows g (sc[i][0..1]) and g + 8 (sc[i][2..3]), keys j0 + 8i + 2t, +1
            const bool masked = j0 + kTK - 1 > pos_lo;
            float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
            for (int i = 0; i < kTK / 8; ++i) {
                const int j = j0 + 8 * i + 2 * t;
                const float relA = (float)(j - posA), relB = (float)(j - posB);
                sc[i][0] = fmaf(sc[i][0], qscale, slope2 * relA);
                sc[i][1] = fmaf(sc[i][1], qscale, slope2 * (relA + 1.f));
                sc[i][2] = fmaf(sc[i][2], qscale, slope2 * relB);
                sc[i][3] = fmaf(sc[i][3], qscale, slope2 * (relB + 1.f));
                if (masked) {
                    sc[i][0] = j <= posA ? sc[i][0] : -INFINITY;
                    sc[i][1] = j + 1 <= posA ? sc[i][1] : -INFINITY;
                    sc[i][2] = j <= posB ? sc[i][2] : -INFINITY;
                    sc[i][3] = j + 1 <= posB ? sc[i][3] : -INFINITY;
                }
                mxA = fmaxf(mxA, fmaxf(sc[i][0], sc[i][1]));
                mxB = fmaxf(mxB, fmaxf(sc[i][2], sc[i][3]));
            }
            mxA = fmaxf(mxA, __shfl_xor_sync(kFull, mxA, 1));
            mxA = fmaxf(mxA, __shfl_xor_sync(kFull, mxA, 2));
            mxB = fmaxf(mxB, __shfl_xor_sync(kFull, mxB, 1));
            mxB = fmaxf(mxB, __shfl_xor_sync(kFull, mxB, 2));
            // Key 0 is visible to every row, so after the first tile the running maxima are finite.
            const float mA_new = fmaxf(mA, mxA), mB_new = fmaxf(mB, mxB);
            const float alphaA = ex2(mA - mA_new), alphaB = ex2(mB - mB_new);
            const bool rescale = __any_sync(kFull, mA_new > mA || mB_new > mB);
            mA = mA_new;
            mB = mB_new;

            uint32_t pa[kTK / 16][4];
            float sumA = 0.f, sumB = 0.f;
#pragma unroll
            for (int kk = 0; kk < kTK / 16; ++kk) {
                pa[kk][0] = pack_bf16(ex2(sc[2 * kk][0] - mA_new), ex2(sc[2 * kk][1] - mA_new), sumA);
                pa[kk][1] = pack_bf16(ex2(sc[2 * kk][2] - mB_new), ex2(sc[2 * kk][3] - mB_new), sumB);
                pa[kk][2] = pack_bf16(ex2(sc[2 * kk + 1][0] - mA_new), ex2(sc[2 * kk + 1][1] - mA_new), sumA);
                pa[kk][3] = pack_bf16(ex2(sc[2 * kk + 1][2] - mB_new), ex2(sc[2 * kk + 1][3] - mB_new), sumB);
            }
            lA = fmaf(lA, alphaA, sumA);
            lB = fmaf(lB, alphaB, sumB);
            if (rescale) {
#pragma unroll
                for (int i = 0; i < NT; ++i) {
                    o[i][0] *= alphaA;
                    o[i][1] *= alphaA;
                    o[i][2] *= alphaB;
                    o[i][3] *= alphaB;
                }
            }

            // ---- O[row][dim] += P[row][key] * V[key][dim]; V transposed on the fly by ldmatrix.trans
            {
                const uint32_t vbase = smem_u32(vst);
                const int vrow = lrow + 8 * (lmat & 1);
#pragma unroll
                for (int kk = 0; kk < kTK / 16; ++kk) {
#pragma unroll
                    for (int jj = 0; jj < NT / 2; ++jj) {
                        uint32_t b[4];
                        ldmatrix_x4_trans(b, vbase + swz(16 * kk + vrow, 2 * jj + (lmat >> 1)));
                        mma_bf16(o[2 * jj], pa[kk], b[0], b[1]);
                        mma_bf16(o[2 * jj + 1], pa[kk], b[2], b[3]);
                    }
                }
            }
        }

        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[st]);
    }
    if (!ok) return;

    // ---- denominators over the quad, normalise, store
    lA += __shfl_xor_sync(kFull, lA, 1);
    lA += __shfl_xor_sync(kFull, lA, 2);
    lB += __shfl_xor_sync(kFull, lB, 1);
    lB += __shfl_xor_sync(kFull, lB, 2);
    const float invA = 1.f / lA, invB = 1.f / lB;
    if (validA) {
        uint32_t* oA = reinterpret_cast<uint32_t*>(p.out + ((size_t)(qstart + iA) * p.Hq + h) * D);
#pragma unroll
        for (int i = 0; i < NT; ++i) oA[i * 4 + t] = float2_to_bf16x2(o[i][0] * invA, o[i][1] * invA);
    }
    if (validB) {
        uint32_t* oB = reinterpret_cast<uint32_t*>(p.out + ((size_t)(qstart + iB) * p.Hq + h) * D);
#pragma unroll
        for (int i = 0; i < NT; ++i) oB[i * 4 + t] = float2_to_bf16x2(o[i][2] * invB, o[i][3] * invB);
    }
}

template <int D, int G>
int launch_one(const CUtensorMap& mk, const CUtensorMap& mv, const PrefillParams& p, int B, int max_q_len,
               cudaStream_t stream) {
    using C = PrefillCfg<D>;
    static std::atomic<bool> configured[kMaxDevices];
    if (!ensure_smem_limit(prefill_kernel<D, G>, C::SMEM, configured)) return OPT_GQA_ERR_CUDA;
    constexpr int TQ = kRows / G;
    dim3 grid((max_q_len + TQ - 1) / TQ, p.Hkv, B);
    return launch_dependent(prefill_kernel<D, G>, grid, dim3((kConsumers + 1) * 32), C::SMEM, stream, mk, mv, p);
}

template <int D>
int launch_g(const CUtensorMap& mk, const CUtensorMap& mv, const PrefillParams& p, int B, int G, int max_q_len,
             cudaStream_t stream) {
    switch (G) {
        case 1: return launch_one<D, 1>(mk, mv, p, B, max_q_len, stream);
        case 2: return launch_one<D, 2>(mk, mv, p, B, max_q_len, stream);
        case 4: return launch_one<D, 4>(mk, mv, p, B, max_q_len, stream);
        case 8: return launch_one<D, 8>(mk, mv, p, B, max_q_len, stream);
    }
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace

int launch_prefill(void* out, const void* q, const int32_t* q_start_loc, int max_q_len, const void* k_cache,
                   const void* v_cache, const int32_t* block_tables, int max_blocks_per_seq,
                   const int32_t* context_lens, const float* alibi_slopes, float scale, int B, int Hq, int Hkv,
                   int D, int bs, int64_t num_blocks, int* device_status, cudaStream_t stream) {
    const uint64_t rows = (uint64_t)num_blocks * (uint64_t)Hkv * (uint64_t)bs;
    if (rows == 0 || rows > 0x7fffffffull) return OPT_GQA_ERR_SHAPE;
    if (B > 65535 || Hkv > 65535) return OPT_GQA_ERR_SHAPE;
    CUtensorMap mk, mv;
    if (!make_cache_map(&mk, k_cache, rows, D, kSub) || !make_cache_map(&mv, v_cache, rows, D, kSub)) return OPT_GQA_ERR_CUDA;
    PrefillParams p;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.q_start_loc = q_start_loc;
    p.block_tables = block_tables;
    p.context_lens = context_lens;
    p.slopes = alibi_slopes;
    p.status = device_status;
    p.scale = scale;
    p.max_blocks = max_blocks_per_seq;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.bs = bs;
    const int G = Hq / Hkv;
    if (D == 128) return launch_g<128>(mk, mv, p, B, G, max_q_len, stream);
    if (D == 64) return launch_g<64>(mk, mv, p, B, G, max_q_len, stream);
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace optgqa

// Q/K/V projection of Eq. 1 for the tokens of one decode step, with the three weight matrices stored
// side by side as one 4-bit group-quantised matrix W [K, N] (N = (Hq + 2 Hkv) D), and the keys and
// values written straight into the paged cache (Algorithm 1, "Reshape and store K, V into C_K, C_V").
//
// The step is a matrix-vector product per token: every weight is read once and used T times, so for the
// few tokens of a decode step the floor is the HBM read of the codes (half a byte per weight); what the
// kernel has to keep small to get near it is the integer work of turning codes into bf16.
// The product runs on the tensor cores all the same, because unpacking eight codes and multiplying them
// with T activations each on the plain ALUs would cost more issue slots than the memory system leaves:
// the output features are the rows of an m16n8k16 tile, the tokens its eight columns, and the codes go
// from global memory to the A-operand registers without passing through shared memory.
//
// Kernel layout of the weights (written once by int4_prepack_kernel from the interchange layout):
//   wp   uint4 [N/16][K/64][32]   lane l of a warp reads entry [mt][kc][l]: word j (0..3) of it holds the
//                                 eight codes of the lane's A fragment for k-step j of the 64-row chunk kc.
//                                 With r = l/4, c = l%4, blk = j/2, s = j%2 the fragment register i (0..3)
//                                 covers output feature 16 mt + r + 8 (i%2) and the two rows
//                                 k = 64 kc + 32 blk + 8 c + 4 s + 2 (i/2) + e, e = 0, 1; code e sits in
//                                 nibble i + 4 e.  (The rows of a k-step are permuted against the plain
//                                 MMA order so that the matching B fragment of a lane is one 16-byte load
//                                 of eight consecutive activations: a sum over k does not mind the order.)
//   sz   uint32 [K/gs][N]         low half: the scale (bf16); high half: 128 + zero point (bf16)
//
// Codes become bf16 by or-ing them into the mantissa of 128.0 (0x4300): 128 + code, exact; subtracting
// 128 + zero gives code - zero exactly.  The products with the activations are accumulated in fp32 per
// group and the group's scale is applied to the fp32 sum, so no weight is ever rounded.
#include "common.cuh"
#include "tma_mma.cuh"

namespace optgqa {
namespace {

constexpr int kProjWarps = 8;         // warps of a CTA; they split K between them
constexpr int kFeatPerCta = 32;       // output features of a CTA: two m16 tiles
constexpr int kRedStride = 36;        // floats between the tokens' rows of the cross-warp sum (bank spread)
constexpr int kMaxSlices = 4;         // CTAs of a cluster that share a tile, a slice of K each

struct ProjParams {
    const uint16_t* x;       // [T, K] bf16
    const uint4* wp;
    const uint32_t* sz;
    uint16_t* q_out;         // [T, Hq D]
    uint16_t* k_out;         // [T, Hkv D] or null
    uint16_t* v_out;
    uint16_t* k_cache;       // paged pool or null
    uint16_t* v_cache;
    const int64_t* slot_mapping;
    int T, K, N, Hq, Hkv, D, bs;
    long long num_blocks;
    int whole_ctas;          // CTAs 0 .. whole_ctas - 1 take a tile each; the rest share the remaining tiles, a cluster per tile
};

__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// 128 + code for the two codes in nibbles `shift/4` and `shift/4 + 4` of w, as a bf16 pair.
// (One three-input logic instruction: (a & mask) | magic.  Written out because the compiler otherwise spends two.)
__device__ __forceinline__ uint32_t codes_to_bf16x2(uint32_t w, int shift) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(w >> shift), "r"(0x000F000Fu), "r"(0x43004300u));
    return d;
}

__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// Rounds the sums of features n, n + 1 of token t to bf16 and stores them where they belong: the query output, the
// plain key/value outputs, the paged cache at the token's slot.
__device__ __forceinline__ void store_pair(const ProjParams& p, int t, int n, float s0, float s1) {
    const uint32_t pair = (uint32_t)float_to_bf16_bits(s0) | ((uint32_t)float_to_bf16_bits(s1) << 16);
    const int qn = p.Hq * p.D, kvn = p.Hkv * p.D;
    if (n < qn) {
        *reinterpret_cast<uint32_t*>(p.q_out + (size_t)t * qn + n) = pair;
        return;
    }
    const bool is_k = n < qn + kvn;
    const int col = n - qn - (is_k ? 0 : kvn);
    uint16_t* plain = is_k ? p.k_out : p.v_out;
    uint16_t* cache = is_k ? p.k_cache : p.v_cache;
    if (plain) *reinterpret_cast<uint32_t*>(plain + (size_t)t * kvn + col) = pair;
    if (cache) {
        const long long slot = p.slot_mapping[t];
        const long long page = slot / p.bs;
        if (slot >= 0 && page < p.num_blocks) {
            const int h = col / p.D, d = col % p.D;
            const size_t dst = (((size_t)page * p.Hkv + h) * p.bs + (size_t)(slot % p.bs)) * p.D + d;
            *reinterpret_cast<uint32_t*>(cache + dst) = pair;
        }
    }
}

// Thread-block cluster: this CTA's rank and the cluster's size, the cluster-wide barrier, and a store to the same
// shared-memory location in another CTA of the cluster.
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_float2(const void* local_smem, uint32_t rank, float2 v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local_smem)), "r"(rank));
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(remote), "f"(v.x), "f"(v.y) : "memory");
}

// NT: token tiles of eight per CTA; CPG: 64-row chunks per quantisation group.
//
// One CTA per 32-feature tile leaves a last, short wave: N / 32 tiles rarely divide by the CTAs the GPU holds, and a
// tile's CTA is a chain of K / 64 / 8 chunks per warp whatever else runs.  The launch therefore gives whole tiles only
// to as many CTAs as fill complete waves (p.whole_ctas); each remaining tile goes to a cluster whose CTAs take a
// slice of K each, so that the tail is a fraction as long, and add their partial sums up through distributed shared
// memory (rank order, so the result does not depend on timing).
template <int NT, int CPG>
__global__ void __launch_bounds__(kProjWarps * 32, 2) qkv_int4_kernel(const ProjParams p) {
    constexpr int PF = NT == 1 ? 4 : 2;   // chunks in flight per warp; a multiple of CPG
    static_assert(PF % CPG == 0, "ring must hold whole groups");
    constexpr int GSLOTS = PF / CPG;
    __shared__ float red[kProjWarps][8 * NT][kRedStride];
    __shared__ __align__(8) float recv[kMaxSlices][8 * NT][kRedStride];   // K slices' sums, written by the cluster's CTAs

    grid_dependency_launch();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = lane >> 2, c = lane & 3;
    const int KC = p.K >> 6;
    // the CTA's tile and its slice of the tile's quantisation groups; the warps split the slice
    const bool sliced = (int)blockIdx.x >= p.whole_ctas;
    const int csize = sliced ? (int)cluster_size() : 1, crank = sliced ? (int)cluster_rank() : 0;
    const int tile = sliced ? p.whole_ctas + ((int)blockIdx.x - p.whole_ctas) / csize : (int)blockIdx.x;
    const int tile_groups = KC / CPG;
    const int g0 = tile_groups * crank / csize, groups = tile_groups * (crank + 1) / csize - g0;
    const int gpw = (groups + kProjWarps - 1) / kProjWarps;
    const int kc0 = (g0 + min(groups, warp * gpw)) * CPG;
    const int kc1 = (g0 + min(groups, (warp + 1) * gpw)) * CPG;
    const int n0 = tile * kFeatPerCta;
    const int t0 = blockIdx.y * 8 * NT;

    const uint4* w0 = p.wp + (size_t)(2 * tile) * KC * 32 + lane;
    const uint4* w1 = w0 + (size_t)KC * 32;
    const uint4* xrow[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int t = min(t0 + nt * 8 + r, p.T - 1);   // rows past T repeat the last token; never stored
        xrow[nt] = reinterpret_cast<const uint4*>(p.x + (size_t)t * p.K) + c;
    }
    const uint32_t* szcol = p.sz + n0 + r;

    uint4 W[PF][2];
    uint4 X[PF][NT][2];
    uint32_t SZ[GSLOTS][4];
    auto fetch_w = [&](int u, int kc) {
        W[u][0] = __ldcs(w0 + (size_t)kc * 32);
        W[u][1] = __ldcs(w1 + (size_t)kc * 32);
        if (u % CPG == 0) {
            const uint32_t* s = szcol + (size_t)(kc / CPG) * p.N;
#pragma unroll
            for (int i = 0; i < 4; ++i) SZ[u / CPG][i] = __ldg(s + 8 * i);
        }
    };
    auto fetch_x = [&](int u, int kc) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            X[u][nt][0] = __ldcg(xrow[nt] + kc * 8);
            X[u][nt][1] = __ldcg(xrow[nt] + kc * 8 + 4);
        }
    };

    float acc[2][NT][4], part[2][NT][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[m][nt][i] = 0.f;

    // the first weights are requested before the preceding kernel of the stream has finished: they do not
    // depend on it, only the activations do
#pragma unroll
    for (int u = 0; u < PF; ++u)
        if (kc0 + u < kc1) fetch_w(u, kc0 + u);
    grid_dependency_wait();
#pragma unroll
    for (int u = 0; u < PF; ++u)
        if (kc0 + u < kc1) fetch_x(u, kc0 + u);

    uint32_t zpair[4];
    float scale[4];
    for (int kc = kc0; kc < kc1; kc += PF) {
#pragma unroll
        for (int u = 0; u < PF; ++u) {
            if (kc + u >= kc1) break;
            if (u % CPG == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t s = SZ[u / CPG][i];
                    zpair[i] = __byte_perm(s, s, 0x3232);
                    scale[i] = __uint_as_float(s << 16);
                }
#pragma unroll
                for (int m = 0; m < 2; ++m)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) part[m][nt][i] = 0.f;
            }
            const uint32_t wj[2][4] = {{W[u][0].x, W[u][0].y, W[u][0].z, W[u][0].w},
                                       {W[u][1].x, W[u][1].y, W[u][1].z, W[u][1].w}};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int m = 0; m < 2; ++m) {
                    uint32_t a[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        a[i] = sub_bf16x2(codes_to_bf16x2(wj[m][j], 4 * i), zpair[2 * m + (i & 1)]);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint4 xv = X[u][nt][j >> 1];
                        if (j & 1) mma_bf16(part[m][nt], a, xv.z, xv.w);
                        else mma_bf16(part[m][nt], a, xv.x, xv.y);
                    }
                }
            }
            if (kc + u + PF < kc1) {
                fetch_w(u, kc + u + PF);
                fetch_x(u, kc + u + PF);
            }
            if (u % CPG == CPG - 1) {
#pragma unroll
                for (int m = 0; m < 2; ++m)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            acc[m][nt][i] = fmaf(scale[2 * m + (i >> 1)], part[m][nt][i], acc[m][nt][i]);
            }
        }
    }

    // cross-warp sum in a fixed order: red[warp][token][feature]
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                red[warp][nt * 8 + 2 * c + (i & 1)][16 * m + r + 8 * (i >> 1)] = acc[m][nt][i];
    __syncthreads();

    // one thread per (token, pair of features): 16 pairs x 8 NT tokens
    static_assert(16 * 8 * NT <= kProjWarps * 32, "the epilogue needs a thread per output pair");
    const int tl = threadIdx.x >> 4, f = (threadIdx.x & 15) * 2;
    float s0 = 0.f, s1 = 0.f;
    if (threadIdx.x < 16 * 8 * NT) {
#pragma unroll
        for (int w = 0; w < kProjWarps; ++w) {
            s0 += red[w][tl][f];
            s1 += red[w][tl][f + 1];
        }
    }
    if (!sliced) {
        if (threadIdx.x < 16 * 8 * NT && t0 + tl < p.T) store_pair(p, t0 + tl, n0 + f, s0, s1);
        return;
    }
    // a K slice: CTA o of the cluster finishes an equal share of the outputs; every CTA writes its sums for that
    // share into slot `crank` of o's shared memory, and after one cluster barrier each CTA adds up what it received,
    // in rank order.  (Nothing touches another CTA's shared memory after the barrier, so a CTA may end at once.)
    const int share = 16 * 8 * NT / csize;
    if (threadIdx.x < 16 * 8 * NT)
        st_cluster_float2(&recv[crank][tl][f], (uint32_t)(threadIdx.x / share), make_float2(s0, s1));
    cluster_sync_all();
    if ((int)threadIdx.x < share) {
        const int idx = crank * share + threadIdx.x;
        const int tk = idx >> 4, fk = (idx & 15) * 2;
        float t_0 = 0.f, t_1 = 0.f;
        for (int k = 0; k < csize; ++k) {
            const float2 v = *reinterpret_cast<const float2*>(&recv[k][tk][fk]);
            t_0 += v.x;
            t_1 += v.y;
        }
        if (t0 + tk < p.T) store_pair(p, t0 + tk, n0 + fk, t_0, t_1);
    }
}

// One thread per uint4 of wp, and (second part of the grid-stride range) one per entry of sz.
__global__ void __launch_bounds__(256)
int4_prepack_kernel(uint4* __restrict__ wp, uint32_t* __restrict__ sz, const uint32_t* __restrict__ qweight,
                    const uint16_t* __restrict__ scales, const uint32_t* __restrict__ qzeros, int K, int N, int gs) {
    const long long n_wp = (long long)(N / 16) * (K / 64) * 32;
    const long long n_sz = (long long)(K / gs) * N;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < n_wp) {
        const int lane = (int)(idx & 31);
        const long long tile = idx >> 5;
        const int kc = (int)(tile % (K / 64));
        const int mt = (int)(tile / (K / 64));
        const int r = lane >> 2, c = lane & 3;
        uint32_t out[4];
        for (int j = 0; j < 4; ++j) {
            const int blk = j >> 1, s = j & 1;
            const int qrow = 8 * kc + 4 * blk + c;                 // word row of qweight: rows 8 qrow .. 8 qrow + 7
            const uint32_t lo = qweight[(size_t)qrow * N + 16 * mt + r];
            const uint32_t hi = qweight[(size_t)qrow * N + 16 * mt + r + 8];
            uint32_t w = 0;
            for (int i = 0; i < 4; ++i) {
                const uint32_t src = (i & 1) ? hi : lo;
                for (int e = 0; e < 2; ++e) {
                    const int within = 4 * s + 2 * (i >> 1) + e;   // row inside the word
                    w |= ((src >> (4 * within)) & 0xFu) << (4 * (i + 4 * e));
                }
            }
            out[j] = w;
        }
        wp[idx] = make_uint4(out[0], out[1], out[2], out[3]);
    } else if (idx < n_wp + n_sz) {
        const long long e = idx - n_wp;
        const int n = (int)(e % N);
        const int g = (int)(e / N);
        const uint32_t zero = (qzeros[(size_t)g * (N / 8) + n / 8] >> (4 * (n % 8))) & 0xFu;
        // bf16 of 128 + zero: 0x4300 with the zero point in the low mantissa bits
        sz[e] = (uint32_t)scales[e] | ((0x4300u | zero) << 16);
    }
}

constexpr int kSliceCtas = kMaxSlices;        // CTAs of a cluster: K slices of a tail tile

// Launches the projection for `tiles` feature tiles and `chunks` passes over the tokens.  With one pass, the tiles
// beyond the last complete wave of CTAs (as many clusters as the GPU holds at once) are cut into kSliceCtas slices of
// K each, unless they are more than half a wave: then, or when the slices would not hold a group each, every tile
// keeps its own CTA.
template <int NT, int CPG>
int launch_proj(ProjParams p, int tiles, int chunks, cudaStream_t stream) {
    static std::atomic<int> wave_ctas[kMaxDevices];       // 0: not asked yet
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kProjWarps * 32);
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kSliceCtas;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;

    int wave = 0, dev = 0;
    if (chunks == 1 && (p.K >> 6) / CPG >= kSliceCtas && cudaGetDevice(&dev) == cudaSuccess) {
        const bool cached = dev >= 0 && dev < kMaxDevices;
        wave = cached ? wave_ctas[dev].load(std::memory_order_acquire) : 0;
        if (wave == 0) {
            cfg.gridDim = dim3(kSliceCtas);
            cfg.numAttrs = 2;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, qkv_int4_kernel<NT, CPG>, &cfg) != cudaSuccess) clusters = 0;
            wave = clusters > 0 ? clusters * kSliceCtas : -1;
            if (cached) wave_ctas[dev].store(wave, std::memory_order_release);
        }
    }
    const int tail = wave > 0 ? tiles % wave : 0;
    if (tail > 0 && tiles > wave && 2 * tail <= wave) {
        p.whole_ctas = tiles - tail;
        cfg.gridDim = dim3((unsigned)(p.whole_ctas + tail * kSliceCtas), (unsigned)chunks);
        cfg.numAttrs = 2;
    } else {
        p.whole_ctas = tiles;
        cfg.gridDim = dim3((unsigned)tiles, (unsigned)chunks);
        cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, qkv_int4_kernel<NT, CPG>, p) == cudaSuccess ? OPT_GQA_OK : OPT_GQA_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool proj_shape_ok(int K, int N, int gs) {
    return K > 0 && N > 0 && (gs == 64 || gs == 128) && K % gs == 0 && N % kFeatPerCta == 0;
}

}  // namespace
}  // namespace optgqa

using namespace optgqa;

extern "C" size_t opt_gqa_int4_packed_bytes(int K, int N, int gs) {
    if (!proj_shape_ok(K, N, gs)) return 0;
    return (size_t)K * N / 2 + (size_t)(K / gs) * N * 4;
}

extern "C" int opt_gqa_int4_prepack(void* packed, const uint32_t* qweight, const void* scales,
                                    const uint32_t* qzeros, int K, int N, int gs, void* stream) {
    if (!proj_shape_ok(K, N, gs)) return OPT_GQA_ERR_SHAPE;
    if (!packed || !qweight || !scales || !qzeros) return OPT_GQA_ERR_NULL;
    if (!aligned16(packed)) return OPT_GQA_ERR_ALIGN;
    uint4* wp = static_cast<uint4*>(packed);
    uint32_t* sz = reinterpret_cast<uint32_t*>(static_cast<char*>(packed) + (size_t)K * N / 2);
    const long long total = (long long)(N / 16) * (K / 64) * 32 + (long long)(K / gs) * N;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return OPT_GQA_ERR_SHAPE;
    int4_prepack_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        wp, sz, qweight, static_cast<const uint16_t*>(scales), qzeros, K, N, gs);
    return cudaGetLastError() == cudaSuccess ? OPT_GQA_OK : OPT_GQA_ERR_CUDA;
}

extern "C" int opt_gqa_qkv_project_int4(void* q_out, void* k_out, void* v_out, void* k_cache, void* v_cache,
                                        const int64_t* slot_mapping, const void* x, const void* packed, int T, int K,
                                        int Hq, int Hkv, int D, int bs, int64_t num_blocks, int gs, void* stream) {
    if (T < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || (D != 64 && D != 128)) return OPT_GQA_ERR_SHAPE;
    const long long Nl = (long long)(Hq + 2 * Hkv) * D;
    if (Nl > 0x7fffffffLL || !proj_shape_ok(K, (int)Nl, gs)) return OPT_GQA_ERR_SHAPE;
    const bool to_cache = k_cache || v_cache;
    if (to_cache && ((bs != 16 && bs != 32) || num_blocks <= 0)) return OPT_GQA_ERR_SHAPE;
    if (T == 0) return OPT_GQA_OK;
    if (!q_out || !x || !packed) return OPT_GQA_ERR_NULL;
    if ((k_cache == nullptr) != (v_cache == nullptr) || (k_out == nullptr) != (v_out == nullptr)) return OPT_GQA_ERR_NULL;
    if (!to_cache && !k_out) return OPT_GQA_ERR_NULL;
    if (to_cache && !slot_mapping) return OPT_GQA_ERR_NULL;
    if (!aligned16(q_out) || !aligned16(x) || !aligned16(packed) || !aligned16(k_out) || !aligned16(v_out) ||
        !aligned16(k_cache) || !aligned16(v_cache))
        return OPT_GQA_ERR_ALIGN;
    ProjParams p;
    p.x = static_cast<const uint16_t*>(x);
    p.wp = static_cast<const uint4*>(packed);
    p.sz = reinterpret_cast<const uint32_t*>(static_cast<const char*>(packed) + (size_t)K * Nl / 2);
    p.q_out = static_cast<uint16_t*>(q_out);
    p.k_out = static_cast<uint16_t*>(k_out);
    p.v_out = static_cast<uint16_t*>(v_out);
    p.k_cache = static_cast<uint16_t*>(k_cache);
    p.v_cache = static_cast<uint16_t*>(v_cache);
    p.slot_mapping = slot_mapping;
    p.T = T; p.K = K; p.N = (int)Nl; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.bs = bs;
    p.num_blocks = num_blocks;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int NT = T <= 8 ? 1 : 2;
    const long long chunks = ((long long)T + 8 * NT - 1) / (8 * NT);
    if (chunks > 65535) return OPT_GQA_ERR_SHAPE;
    const int tiles = (int)(Nl / kFeatPerCta);
    if (NT == 1) return gs == 64 ? launch_proj<1, 1>(p, tiles, (int)chunks, cs) : launch_proj<1, 2>(p, tiles, (int)chunks, cs);
    return gs == 64 ? launch_proj<2, 1>(p, tiles, (int)chunks, cs) : launch_proj<2, 2>(p, tiles, (int)chunks, cs);
}

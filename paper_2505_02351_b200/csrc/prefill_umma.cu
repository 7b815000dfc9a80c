// Multi-token (chunked-prefill) GQA-ALiBi attention over the paged cache on the 5th-generation
// tensor cores: tcgen05.mma with accumulators in tensor memory (the prompt branch of Algorithms 1
// and 2 with "Create ALiBi bias" and the causal mask; Eq. 3-5).  bf16, head_dim 128.
//
// One CTA per (query block, KV head, sequence).  The G query heads of the group times TQ = 128 / G
// consecutive new tokens are the 128 rows of the CTA's tiles, so every K/V tile is fetched once for
// the whole group ("Shared Key-Value").  Six warps, three roles:
//   warps 0-3  one thread per row: read the row of the 128 x kTN score tile S from tensor memory (it
//              already holds the ALiBi term slope_h*(j - j0) of Eq. 3 relative to the tile's first
//              key j0; the rest of the term is a constant of the row and tile), mask j > pos from the
//              indices, keep the row's running maximum and denominator (Eq. 4, online; two passes
//              over the scores in registers, first the maximum, then p), write p as bf16 back into
//              tensor memory over S, rescale O when the maximum moved, and store the normalised rows
//   warp 4     producer: walks the block table and fetches kTN-key K and V tiles (2-D TMA boxes of
//              16 token rows x 128 bytes, 128-byte swizzle) into a ring, plus the Q tile
//   warp 5     one thread issues S = Q K^T (operands in shared memory) and O += P V (P from tensor
//              memory, V in shared memory addressed MN-major) and commits them to mbarriers
// S is double-buffered in tensor memory, so the tensor core works on tile j+1's scores and tile
// j-1's P V while the row threads do tile j's softmax.  Tiles are taken from the diagonal backwards
// (nearest keys first): the ALiBi term falls with distance, so a row's maximum is set by the first
// tiles it sees and O is rescaled only when the maximum still grows by more than 2^8 -- in forward
// order the bias alone would move it every tile.  The ALiBi term inside a tile is added by the tensor core
// itself (a ninth k-step, see kOffQx), so a row thread spends one max per two scores in the first pass and one
// packed FMA, two exp2, one packed add and one conversion per two scores in the second.  The default shape is
// 64-key tiles in a two-stage ring: two CTAs fit on an SM (102 KiB of shared memory and 256 tensor-memory
// columns each) and one CTA's row warps run while the other's wait.
// Every wait is a bounded mbarrier wait.
#include "tma_mma.cuh"

namespace optgqa {

namespace {

constexpr int kRows = 128;         // rows of the CTA's tiles (G heads x TQ tokens)
constexpr int kTN = 64;            // keys per tile
constexpr int kSub = 16;           // token rows per TMA box
constexpr int kKvStages = 2;       // (the issuing thread selects a stage's descriptors with one compare: two stages)
constexpr int kCtasPerSm = 2;
constexpr int kThreads = 192;
constexpr unsigned kFull = 0xffffffffu;
constexpr float kRescaleThreshold = 8.f;   // log2 units: O is rescaled only when a row's maximum grew by more

constexpr int kHalfBytes = kTN * 128;              // one 64-dim column half of a K or V tile (kTN rows of 128 B)
constexpr int kQHalfBytes = kRows * 128;           // one 64-dim column half of the Q tile: 16 KiB
// The ALiBi term rides on the tensor core as one more k-step of S = Q K^T: an extension of Q that holds
// slope_h / |scale| split over three bf16 values, against an extension of K that holds the key's index inside
// the tile three times.  Both are 16-dim K-major operands without swizzle: 8-row x 16-byte core matrices of
// 128 contiguous bytes, the two 8-dim halves of a row group 128 bytes apart, row groups 256 bytes apart.
constexpr int kExtRowGroupBytes = 256;
constexpr int kQxBytes = kRows / 8 * kExtRowGroupBytes;   // 4 KiB
constexpr int kKpBytes = kTN / 8 * kExtRowGroupBytes;     // 2 KiB
// barriers: q_full, k_full[], k_empty[], v_full[], v_empty[], s_full[2], p_full[2]; then the TMEM base word
constexpr int kNumBars = 1 + 4 * kKvStages + 4;

// Shared memory of a CTA for head dimension D (64 or 128): the Q tile and the K/V rings as D / 64 column halves of
// 128-byte rows, the extension operands, the barriers.
template <int D>
struct PfLayout {
    static constexpr int kHalves = D / 64;
    static constexpr int kTileBytes = kHalves * kHalfBytes;         // a K or V tile
    static constexpr int kQBytes = kHalves * kQHalfBytes;
    static constexpr int kOffQ = 0;
    static constexpr int kOffK = kQBytes;
    static constexpr int kOffV = kOffK + kKvStages * kTileBytes;
    static constexpr int kOffQx = kOffV + kKvStages * kTileBytes;
    static constexpr int kOffKp = kOffQx + kQxBytes;
    static constexpr int kOffBar = kOffKp + kKpBytes;
    static constexpr int kSmemBytes = kOffBar + kNumBars * 8 + 16 + 1024;   // + slack to align the tiles to 1 KiB
};

// tensor-memory columns (fp32 accumulators, 128 lanes each)
constexpr uint32_t kColS = 0;       // S buffers at 0 and kTN; P (bf16 pairs) overlays the first kTN / 2 columns of its S
constexpr uint32_t kColO = 2 * kTN;                       // D columns
constexpr uint32_t kTmemCols = 256;                       // a power of two >= 2 kTN + 128

struct UmmaParams {
    __nv_bfloat16* out;
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
    int window;             // > 0: token at pos sees keys pos - window < j <= pos only
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Arrives on `bar` once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// Shared-memory matrix descriptor: 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

// Shared-memory matrix descriptor without swizzle (core matrices of 8 rows x 16 bytes): lbo = distance between the
// core matrices of one row group along K, sbo = distance between row groups.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46);
}

// The descriptor of the same layout `bytes` further on in shared memory (a multiple of 16; the address field counts
// 16-byte units and shared memory ends below 2^18, so only the low word changes): one add where building a
// descriptor anew costs several instructions of the one thread that issues all tensor-core work.
__device__ __forceinline__ uint64_t desc_advance(uint64_t desc, uint32_t bytes) {
    return (desc & 0xFFFFFFFF00000000ull) | (uint32_t)((uint32_t)desc + (bytes >> 4));
}

// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M = 128, N = n, A K-major (optionally negated), B K-major
// or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major, uint32_t n, bool negate_a = false) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((negate_a ? 1u : 0u) << 13) | ((b_mn_major ? 1u : 0u) << 16) |
           ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}

// Starts the load of 32 consecutive 32-bit columns of this thread's lane; the registers are valid only after
// tmem_wait_ld() (and tmem_pin(), which keeps the compiler from moving their uses above the wait).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_pin(uint32_t* r) {     // 32 registers, no instruction
#pragma unroll
    for (int i = 0; i < 32; i += 16)
        asm volatile("" : "+r"(r[i]), "+r"(r[i + 1]), "+r"(r[i + 2]), "+r"(r[i + 3]), "+r"(r[i + 4]), "+r"(r[i + 5]),
                          "+r"(r[i + 6]), "+r"(r[i + 7]), "+r"(r[i + 8]), "+r"(r[i + 9]), "+r"(r[i + 10]), "+r"(r[i + 11]),
                          "+r"(r[i + 12]), "+r"(r[i + 13]), "+r"(r[i + 14]), "+r"(r[i + 15])
                     :
                     : "memory");
}

// 32 consecutive fp32 columns of this thread's lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    tmem_ld32_issue(taddr, r);
    tmem_wait_ld();
    tmem_pin(r);
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
          "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
          "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// max of three (one instruction on sm_100)
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Pass 1 over one 32-key chunk of a row's raw scores s = q.k + (slope/scale)*(key index in the tile): running
// maxima.  The map to log2 units, t = s*qscale + (tile constant), is increasing, so it is applied to the maximum
// afterwards.  kMasked adds the select of the visible keys, lo < key <= pos (causal bound pos; lo = pos - window,
// or -1); tiles strictly inside that range skip it.
template <bool kMasked>
__device__ __forceinline__ void chunk_max(const float (&v)[32], int key0, int pos, int lo, float (&mx)[4]) {
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        float s0 = v[e], s1 = v[e + 1];
        if (kMasked) {
            s0 = (key0 + e <= pos && key0 + e > lo) ? s0 : -INFINITY;
            s1 = (key0 + e + 1 <= pos && key0 + e + 1 > lo) ? s1 : -INFINITY;
        }
        mx[(e >> 1) & 3] = max3(mx[(e >> 1) & 3], s0, s1);
    }
}

// Two fp32 values in one 64-bit register, for the packed fp32 instructions of sm_100 (one issue slot for two lanes).
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Pass 2 over one chunk: p = 2^(s*qscale + bias) with the tile's ALiBi constant and the row maximum folded into
// bias; bf16 pairs for the tensor core; returns the chunk's sum of p.
template <bool kMasked>
__device__ __forceinline__ float chunk_exp(const float (&v)[32], float qscale, float bias, int key0, int pos, int lo,
                                           uint32_t (&w)[16]) {
    if (kMasked) {
        float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            float t0 = fmaf(v[2 * e], qscale, bias);
            float t1 = fmaf(v[2 * e + 1], qscale, bias);
            t0 = (key0 + 2 * e <= pos && key0 + 2 * e > lo) ? t0 : -INFINITY;
            t1 = (key0 + 2 * e + 1 <= pos && key0 + 2 * e + 1 > lo) ? t1 : -INFINITY;
            const float p0 = ex2(t0), p1 = ex2(t1);
            sm[e & 3] += p0 + p1;
            w[e] = pack2(p0, p1);
        }
        return (sm[0] + sm[1]) + (sm[2] + sm[3]);
    }
    const uint64_t qs2 = pack_f2(qscale, qscale), b2 = pack_f2(bias, bias);
    uint64_t sm2[2] = {pack_f2(0.f, 0.f), pack_f2(0.f, 0.f)};
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const uint64_t t2 = fma2(pack_f2(v[2 * e], v[2 * e + 1]), qs2, b2);
        float t0, t1;
        unpack_f2(t2, t0, t1);
        const float p0 = ex2(t0), p1 = ex2(t1);
        sm2[e & 1] = add2(sm2[e & 1], pack_f2(p0, p1));
        w[e] = pack2(p0, p1);
    }
    float s0, s1;
    unpack_f2(add2(sm2[0], sm2[1]), s0, s1);
    return s0 + s1;
}

// kPaged: K/V come from the paged cache through block_tables (2-D maps over [rows, D]); otherwise from contiguous
// k, v [tokens, Hkv, D] holding exactly the new tokens (3-D maps; the prompt branch with empty caches, where a
// sequence's context is its own new tokens).
template <int D, int G, bool kPaged>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
prefill_umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const UmmaParams p) {
    using L = PfLayout<D>;
    constexpr int kTileBytes = L::kTileBytes, kOffQ = L::kOffQ, kOffK = L::kOffK, kOffV = L::kOffV, kOffQx = L::kOffQx,
                  kOffKp = L::kOffKp;
    constexpr int TQ = kRows / G;     // new tokens per query block
    extern __shared__ char smem_raw[];
    char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kOffBar);
    uint64_t* q_full = bars;
    uint64_t* k_full = bars + 1;
    uint64_t* k_empty = k_full + kKvStages;
    uint64_t* v_full = k_empty + kKvStages;
    uint64_t* v_empty = v_full + kKvStages;
    uint64_t* s_full = v_empty + kKvStages;
    uint64_t* p_full = s_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kNumBars);

    grid_dependency_launch();
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
    const int n = kPaged ? p.context_lens[s] : qlen;
    const int i_last = min(qlen, (qb + 1) * TQ) - 1;        // last valid new token of this block
    const int pos_last = n - qlen + i_last;                 // its position; the block sees keys 0 .. pos_last
    // Tiles tile_lo .. tile_hi hold the keys the block sees: up to pos_last, and with a local window no further
    // back than window - 1 keys before the block's first token.
    const int tile_hi = pos_last / kTN;
    const int pos_first = n - qlen + qb * TQ;
    const int tile_lo = p.window > 0 ? max(0, pos_first - p.window + 1) / kTN : 0;
    const int ntiles = tile_hi - tile_lo + 1;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
#pragma unroll
        for (int i = 0; i < kKvStages; ++i) {
            mbar_init(&k_full[i], 1);
            mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1);
            mbar_init(&v_empty[i], 1);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i], kRows);
        }
        tmem_slot[1] = 0;       // set by mbar_wait's callers when a wait gave up (see the end of the kernel)
        fence_barrier_init();
    }
    // The scale may have any sign.  The tensor core multiplies with |scale| in mind: a negative scale negates Q in
    // the instruction (so that the row maximum can still be taken on the raw scores), a zero scale leaves the dot
    // products out altogether and the scores are the bias alone.
    const float sabs = p.scale == 0.f ? 1.f : fabsf(p.scale);
    // Extension operands of the ALiBi k-step (see kOffQx): row r of Q's holds slope_h / |scale| as a sum of three
    // bf16 values, row e of K's the index e three times; dims 3..15 are zero.  With a zero scale the step also
    // runs without slopes (all-zero rows): it is then what initialises the score tile.
    const bool alibi = p.slopes != nullptr || p.scale == 0.f;
    if (alibi) {
        if (threadIdx.x < kRows) {
            const int r = threadIdx.x;
            const float a = p.slopes ? p.slopes[kvh * G + r % G] / sabs : 0.f;
            const __nv_bfloat16 a0 = __float2bfloat16_rn(a);
            const __nv_bfloat16 a1 = __float2bfloat16_rn(a - __bfloat162float(a0));
            const __nv_bfloat16 a2 = __float2bfloat16_rn(a - __bfloat162float(a0) - __bfloat162float(a1));
            char* row = smem + kOffQx + (r >> 3) * kExtRowGroupBytes + (r & 7) * 16;
            *reinterpret_cast<uint4*>(row) = make_uint4((uint32_t)__bfloat16_as_ushort(a0) | ((uint32_t)__bfloat16_as_ushort(a1) << 16),
                                                        (uint32_t)__bfloat16_as_ushort(a2), 0u, 0u);
            *reinterpret_cast<uint4*>(row + 128) = make_uint4(0u, 0u, 0u, 0u);
        } else {
            for (int e = threadIdx.x - kRows; e < kTN; e += kThreads - kRows) {
                const uint32_t eb = __bfloat16_as_ushort(__float2bfloat16_rn((float)e));      // exact: e < 256
                char* row = smem + kOffKp + (e >> 3) * kExtRowGroupBytes + (e & 7) * 16;
                *reinterpret_cast<uint4*>(row) = make_uint4(eb | (eb << 16), eb, 0u, 0u);
                *reinterpret_cast<uint4*>(row + 128) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        fence_proxy_async();
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dependency_wait();     // the cache may still be receiving this step's appended tokens

    if (warp == 4) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_expect_tx(q_full, L::kQBytes);
#pragma unroll
            for (int hf = 0; hf < L::kHalves; ++hf)
                tma_load_3d(smem + kOffQ + hf * kQHalfBytes, &map_q, 64 * hf, kvh * G, qstart + qb * TQ, q_full);
        }
        const int32_t* table = kPaged ? p.block_tables + (size_t)s * p.max_blocks : nullptr;
        const int sub = lane & 7;                           // lanes 0-7 fetch one 16-token slice each
        auto page_of = [&](int j) -> int {         // j counts processed tiles; the tile is tile_hi - j
            const int tok = (tile_hi - j) * kTN + sub * kSub;
            return (kPaged && lane < 8 && tok < n) ? __ldg(table + tok / p.bs) : -1;
        };
        int page = page_of(0);
        for (int j = 0; j < ntiles; ++j) {
            const int st = j % kKvStages;
            const int page_next = j + 1 < ntiles ? page_of(j + 1) : -1;
            const int j0 = (tile_hi - j) * kTN;
            const int nsub = min(kTN / kSub, (n - j0 + kSub - 1) / kSub);     // slices that hold cached tokens
            const int tok = j0 + sub * kSub;
            const int row = (page * p.Hkv + kvh) * p.bs + tok % p.bs;          // row of the [rows, D] view
            bool ok = true;
            if (j >= kKvStages) ok = mbar_wait(&k_empty[st], ((j / kKvStages) - 1) & 1, p.status);
            if (!__all_sync(kFull, ok)) break;
            if (lane == 0) mbar_expect_tx(&k_full[st], (uint32_t)nsub * L::kHalves * kSub * 128u);
            __syncwarp();
            if (lane < nsub) {
                char* dst = smem + kOffK + st * kTileBytes + sub * (kSub * 128);
#pragma unroll
                for (int hf = 0; hf < L::kHalves; ++hf) {
                    if (kPaged) tma_load_2d(dst + hf * kHalfBytes, &map_k, 64 * hf, row, &k_full[st]);
                    else tma_load_3d(dst + hf * kHalfBytes, &map_k, 64 * hf, kvh, qstart + tok, &k_full[st]);
                }
            }
            if (j >= kKvStages) ok = mbar_wait(&v_empty[st], ((j / kKvStages) - 1) & 1, p.status);
            if (!__all_sync(kFull, ok)) break;
            if (lane == 0) mbar_expect_tx(&v_full[st], (uint32_t)nsub * L::kHalves * kSub * 128u);
            __syncwarp();
            if (lane < nsub) {
                char* dst = smem + kOffV + st * kTileBytes + sub * (kSub * 128);
#pragma unroll
                for (int hf = 0; hf < L::kHalves; ++hf) {
                    if (kPaged) tma_load_2d(dst + hf * kHalfBytes, &map_v, 64 * hf, row, &v_full[st]);
                    else tma_load_3d(dst + hf * kHalfBytes, &map_v, 64 * hf, kvh, qstart + tok, &v_full[st]);
                }
            }
            page = page_next;
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ tensor-core issue (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(false, kTN), idesc_pv = instr_desc(true, D);
            const uint32_t idesc_qk = p.scale < 0.f ? instr_desc(false, kTN, true) : idesc_s;
            const bool dots = p.scale != 0.f;
            // Every descriptor that does not change from tile to tile is built once: Q's for the D / 16 k-steps, the
            // extension operands', and per ring stage those of the K tile's first k-step and the V tile's first 16 keys.
            uint64_t q_desc[D / 16], k_desc0[kKvStages], v_desc0[kKvStages];
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
                q_desc[ks] = smem_desc(smem_u32(smem + kOffQ) + (ks >> 2) * kQHalfBytes + (ks & 3) * 32, 16, 1024);
#pragma unroll
            for (int st = 0; st < kKvStages; ++st) {
                k_desc0[st] = smem_desc(smem_u32(smem + kOffK + st * kTileBytes), 16, 1024);
                v_desc0[st] = smem_desc(smem_u32(smem + kOffV + st * kTileBytes), kHalfBytes, 1024);
            }
            const uint64_t qx_desc = smem_desc_plain(smem_u32(smem + kOffQx), 128, kExtRowGroupBytes);
            const uint64_t kp_desc = smem_desc_plain(smem_u32(smem + kOffKp), 128, kExtRowGroupBytes);
            bool ok = mbar_wait(q_full, 0, p.status);
            // O += P V for tile t: P (bf16 pairs, 8 columns per 16 keys) from tensor memory, V addressed MN-major:
            // 64-dim halves kHalfBytes apart (leading offset), groups of 8 keys 1 KiB apart (stride offset).
            auto issue_pv = [&](int t) -> bool {
                const int st = t % kKvStages, sb = t & 1;
                if (!mbar_wait(&p_full[sb], (t >> 1) & 1, p.status)) return false;
                if (!mbar_wait(&v_full[st], (t / kKvStages) & 1, p.status)) return false;
                tc_fence_after();
                const uint64_t vd = st == 0 ? v_desc0[0] : v_desc0[kKvStages - 1];
                const uint32_t p_tmem = tmem_base + kColS + sb * kTN;
                umma_ts(tmem_base + kColO, p_tmem, vd, idesc_pv, t > 0);
#pragma unroll
                for (int kk = 1; kk < kTN / 16; ++kk)
                    umma_ts(tmem_base + kColO, p_tmem + kk * 8, desc_advance(vd, kk * 2048), idesc_pv, true);
                tc_commit(&v_empty[st]);
                return true;
            };
            for (int j = 0; ok && j < ntiles; ++j) {
                const int st = j % kKvStages, sb = j & 1;
                ok = mbar_wait(&k_full[st], (j / kKvStages) & 1, p.status);
                if (!ok) break;
                tc_fence_after();
                // S = Q K^T: both K-major, 16 dims (32 bytes) per step inside the 128-byte swizzled rows
                const uint64_t kd = st == 0 ? k_desc0[0] : k_desc0[kKvStages - 1];
                const uint32_t s_tmem = tmem_base + kColS + sb * kTN;
                if (dots) {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        umma_ss(s_tmem, q_desc[ks], desc_advance(kd, (ks >> 2) * kHalfBytes + (ks & 3) * 32), idesc_qk, ks > 0);
                }
                if (alibi) umma_ss(s_tmem, qx_desc, kp_desc, idesc_s, dots);
                tc_commit(&s_full[sb]);
                tc_commit(&k_empty[st]);
                if (j >= 1) ok = issue_pv(j - 1);
            }
            if (ok) issue_pv(ntiles - 1);
        }
    } else {
        // ------------------------------------------------------------------ one thread per row: softmax, rescale, store
        const int r = threadIdx.x;                    // row of the tiles = tensor-memory lane
        const int tok = r / G, hg = r % G;            // the Q box is filled head-fastest
        const int i = qb * TQ + tok;                  // new-token index in the sequence
        const bool valid = i < qlen;
        // Rows past the end of the block are computed as copies of the last valid position and never stored.
        const int pos = n - qlen + min(i, i_last);
        const int lo = p.window > 0 ? pos - p.window : -1;       // keys lo < j <= pos are visible
        const int h = kvh * G + hg;
        const float qscale = sabs * kLog2e;       // > 0: the tensor core has taken care of the scale's sign
        const float slope2 = p.slopes ? p.slopes[h] * kLog2e : 0.f;
        const float c_row = -slope2 * (float)pos;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;

        for (int j = 0; j < ntiles; ++j) {
            const int sb = j & 1, j0 = (tile_hi - j) * kTN;
            ok = __all_sync(kFull, mbar_wait(&s_full[sb], (j >> 1) & 1, p.status));
            if (!ok) break;
            tc_fence_after();
            const uint32_t s_addr = lane_addr + kColS + sb * kTN;

            // ---- pass 1: the row's scores for the tile's 128 keys (Eq. 3), only their maximum is kept.  The
            // loops over the four 32-key chunks are not unrolled: with one warp per scheduler the code has to
            // stay inside the instruction cache.
            // Only tiles on the diagonal (and at the far edge of a local window) need the select; the choice is
            // made per warp.
            const bool masked = __any_sync(kFull, j0 + kTN - 1 > pos || j0 <= lo);
            const float bias0 = fmaf(slope2, (float)j0, c_row);       // ALiBi term of the tile's first key
            // the whole row of the tile is read once (both loads in flight together) and kept in registers for
            // both passes
            float v[kTN / 32][32];
            {
                uint32_t raw[kTN / 32][32];
#pragma unroll
                for (int c = 0; c < kTN / 32; ++c) tmem_ld32_issue(s_addr + c * 32, raw[c]);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < kTN / 32; ++c) {
                    tmem_pin(raw[c]);
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[c][e] = __uint_as_float(raw[c][e]);
                }
            }
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < kTN / 32; ++c) {
                if (masked) chunk_max<true>(v[c], j0 + c * 32, pos, lo, mx);
                else chunk_max<false>(v[c], j0 + c * 32, pos, lo, mx);
            }
            // qscale > 0: the largest raw score gives the largest t (and -inf stays -inf)
            const float m_tile = fmaf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), qscale, bias0);

            // ---- running maximum: move it (and rescale l and O) only when it grew by more than the threshold
            // (true for the first tile in which the row sees a key: m_used = -inf until then)
            const bool need = m_tile > m_used + kRescaleThreshold;
            const float m_new = need ? m_tile : m_used;
            const float f = need ? ex2(m_used - m_new) : 1.f;          // 0 the first time
            if (j > 0 && __any_sync(kFull, need)) {
                // O holds tiles 0 .. j-1 once tile j-1's P V has completed
                ok = __all_sync(kFull, mbar_wait(&v_empty[(j - 1) % kKvStages], ((j - 1) / kKvStages) & 1, p.status));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    float v[32];
                    uint32_t w[32];
                    tmem_ld32(lane_addr + kColO + c * 32, v);
#pragma unroll
                    for (int e = 0; e < 32; ++e) w[e] = __float_as_uint(v[e] * f);
                    tmem_st32(lane_addr + kColO + c * 32, w);
                }
            }
            m_used = m_new;
            l *= f;

            // ---- pass 2: p = 2^(s - m) (Eq. 4) from the scores read again, rounded to bf16 pairs over the first
            // 64 columns of S: chunk c's 16 columns of P lie below the S columns still to be read
            // (a row that has not seen a key yet has only -inf scores: subtract 0 so that they give p = 0)
            const float m_sub = m_used == -INFINITY ? 0.f : m_used;
            const float bias_m = bias0 - m_sub;
            // Far from the diagonal the ALiBi term alone puts every score of the tile more than 127 binary orders
            // below the row's reference maximum: 2^(s - m) is then exactly zero in this arithmetic (the exponential
            // flushes results below 2^-126 to zero), for every key of the tile.  Where that holds for all rows of
            // the warp, the exponentials are not evaluated: P is written as zeros, the denominator stays as it is.
            // (The tensor core still multiplies the tile: nothing is skipped there.)
            const bool all_zero = __all_sync(kFull, m_tile - m_used < -127.f);
            if (all_zero) {
                uint32_t w[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) w[e] = 0u;
#pragma unroll
                for (int c = 0; c < kTN / 32; ++c) tmem_st16(s_addr + c * 16, w);
            } else {
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < kTN / 32; ++c) {
                    uint32_t w[16];
                    if (masked) sum += chunk_exp<true>(v[c], qscale, bias_m, j0 + c * 32, pos, lo, w);
                    else sum += chunk_exp<false>(v[c], qscale, bias_m, j0 + c * 32, pos, lo, w);
                    tmem_st16(s_addr + c * 16, w);
                }
                l += sum;
            }

            if (j0 + kTN > n) {
                // Rows past the end of the sequence hold whatever the page held, or stale shared memory where no
                // page exists: zero this thread's V row so that 0 * garbage cannot produce NaN.
                const int st = j % kKvStages;
                ok = __all_sync(kFull, mbar_wait(&v_full[st], (j / kKvStages) & 1, p.status));
                if (!ok) break;
                if (r < kTN && j0 + r >= n) {
                    char* vrow = smem + kOffV + st * kTileBytes + r * 128;
#pragma unroll
                    for (int b = 0; b < L::kHalves; ++b)
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            *reinterpret_cast<uint4*>(vrow + b * kHalfBytes + e * 16) = make_uint4(0, 0, 0, 0);
                    fence_proxy_async();
                }
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&p_full[sb]);
        }

        if (ok) {
            // ---- all tiles accumulated once the last P V has completed: normalise (Eq. 5) and store
            ok = __all_sync(kFull, mbar_wait(&v_empty[(ntiles - 1) % kKvStages], ((ntiles - 1) / kKvStages) & 1, p.status));
        }
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l;
            uint4* orow = reinterpret_cast<uint4*>(p.out + ((size_t)(qstart + i) * p.Hq + h) * D);
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                float v[32];
                tmem_ld32(lane_addr + kColO + c * 32, v);
                if (valid) {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        orow[c * 4 + e] = make_uint4(pack2(v[8 * e] * inv, v[8 * e + 1] * inv),
                                                     pack2(v[8 * e + 2] * inv, v[8 * e + 3] * inv),
                                                     pack2(v[8 * e + 4] * inv, v[8 * e + 5] * inv),
                                                     pack2(v[8 * e + 6] * inv, v[8 * e + 7] * inv));
                }
            }
        }
    }

    // ---- every role is done with tensor memory: give it back.  If a bounded wait gave up somewhere (already
    // recorded in the status word), copies or tensor-core work of this CTA may still be in flight: let them
    // drain for a while before the shared and tensor memory are released.
    if (*reinterpret_cast<volatile int*>(p.status) != 0) tmem_slot[1] = 1;
    tc_fence_before();
    __syncthreads();
    if (tmem_slot[1]) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// q [tokens, Hq, D] as a 3-D tensor; a box is 64 dims x the G heads of a group x 128 / G tokens, i.e. one
// 64-dim half of the CTA's 128 rows, head-fastest.  Tokens past the end of q read as zeros.
bool make_q_map(CUtensorMap* map, const void* q, int tokens, int Hq, int G, int D) {
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)(kRows / G)};
    return make_bf16_map(map, q, 3, dims, strides, box);
}

// k or v [tokens, Hkv, D] as a 3-D tensor; a box is 64 dims x one head x 16 tokens.
bool make_kv_map(CUtensorMap* map, const void* kv, int tokens, int Hkv, int D) {
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)tokens};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hkv * D * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)kSub};
    return make_bf16_map(map, kv, 3, dims, strides, box);
}

template <int D, int G, bool kPaged>
int launch_one(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const UmmaParams& p, int B,
               int max_q_len, cudaStream_t stream) {
    static std::atomic<bool> configured[kMaxDevices];
    constexpr int kSmem = PfLayout<D>::kSmemBytes;
    if (!ensure_smem_limit(prefill_umma_kernel<D, G, kPaged>, kSmem, configured)) return OPT_GQA_ERR_CUDA;
    constexpr int TQ = kRows / G;
    dim3 grid((max_q_len + TQ - 1) / TQ, p.Hkv, B);
    return launch_dependent(prefill_umma_kernel<D, G, kPaged>, grid, dim3(kThreads), kSmem, stream, mq, mk, mv, p);
}

template <int D, bool kPaged>
int launch_g(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const UmmaParams& p, int B, int G,
             int max_q_len, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_one<D, 1, kPaged>(mq, mk, mv, p, B, max_q_len, stream);
        case 2: return launch_one<D, 2, kPaged>(mq, mk, mv, p, B, max_q_len, stream);
        case 4: return launch_one<D, 4, kPaged>(mq, mk, mv, p, B, max_q_len, stream);
        case 8: return launch_one<D, 8, kPaged>(mq, mk, mv, p, B, max_q_len, stream);
    }
    return OPT_GQA_ERR_SHAPE;
}

template <bool kPaged>
int launch_d(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const UmmaParams& p, int B, int G,
             int D, int max_q_len, cudaStream_t stream) {
    if (D == 128) return launch_g<128, kPaged>(mq, mk, mv, p, B, G, max_q_len, stream);
    if (D == 64) return launch_g<64, kPaged>(mq, mk, mv, p, B, G, max_q_len, stream);
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace

// bf16, D = 64 or 128, any scale; window > 0 adds the local mask.
int launch_prefill_umma(void* out, const void* q, const int32_t* q_start_loc, int total_q_tokens, int max_q_len,
                        const void* k_cache, const void* v_cache, const int32_t* block_tables, int max_blocks_per_seq,
                        const int32_t* context_lens, const float* alibi_slopes, float scale, int B, int Hq, int Hkv,
                        int D, int bs, int64_t num_blocks, int window, int* device_status, cudaStream_t stream) {
    const uint64_t rows = (uint64_t)num_blocks * (uint64_t)Hkv * (uint64_t)bs;
    if (rows == 0 || rows > 0x7fffffffull || total_q_tokens <= 0) return OPT_GQA_ERR_SHAPE;
    if (B > 65535 || Hkv > 65535) return OPT_GQA_ERR_SHAPE;
    const int G = Hq / Hkv;
    CUtensorMap mq, mk, mv;
    if (!make_q_map(&mq, q, total_q_tokens, Hq, G, D) || !make_cache_map(&mk, k_cache, rows, D, kSub) ||
        !make_cache_map(&mv, v_cache, rows, D, kSub))
        return OPT_GQA_ERR_CUDA;
    UmmaParams p;
    p.out = static_cast<__nv_bfloat16*>(out);
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
    p.window = window;
    return launch_d<true>(mq, mk, mv, p, B, G, D, max_q_len, stream);
}

// The prompt branch with empty caches: q [tokens, Hq, D], k, v [tokens, Hkv, D] contiguous, causal + ALiBi.
int launch_prompt_umma(void* out, const void* q, const void* k, const void* v, const int32_t* q_start_loc,
                       int total_q_tokens, int max_q_len, const float* alibi_slopes, float scale, int B, int Hq,
                       int Hkv, int D, int* device_status, cudaStream_t stream) {
    if (total_q_tokens <= 0 || B > 65535 || Hkv > 65535) return OPT_GQA_ERR_SHAPE;
    const int G = Hq / Hkv;
    CUtensorMap mq, mk, mv;
    if (!make_q_map(&mq, q, total_q_tokens, Hq, G, D) || !make_kv_map(&mk, k, total_q_tokens, Hkv, D) ||
        !make_kv_map(&mv, v, total_q_tokens, Hkv, D))
        return OPT_GQA_ERR_CUDA;
    UmmaParams p;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.q_start_loc = q_start_loc;
    p.block_tables = nullptr;
    p.context_lens = nullptr;
    p.slopes = alibi_slopes;
    p.status = device_status;
    p.scale = scale;
    p.max_blocks = 0;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.bs = 16;
    p.window = 0;
    return launch_d<false>(mq, mk, mv, p, B, G, D, max_q_len, stream);
}

}  // namespace optgqa

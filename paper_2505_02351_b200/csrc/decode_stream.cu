// Partitioned paged GQA-ALiBi decode attention for bf16 caches on sm_100a, persistent
// streaming form (Algorithm 2, "Compute context attention with caches"; Eq. 3-5; the
// long-sequence partitioning described before Eq. 1).
//
// The streams (sequence, KV head), each ceil(n / 16) tiles of 16 tokens long, are laid end to end and cut
// into one contiguous range per worker at tile granularity, so that every SM streams the same number of
// cache bytes whatever the mix of lengths.  A piece is the part of one context partition that lies inside
// one range; it produces a normalised partial result and its log-sum-exp for all G query heads of the
// group ("Shared Key-Value": a K/V tile is brought on-chip once for the whole group), and the merge
// (reduce.cu) combines the pieces of a stream.  The grid is persistent: every warp is an independent worker
// with a private ring of K/V tiles fetched by 2-D TMA (128-byte swizzle) and streams its pieces back to
// back, so the ring never drains between pieces: page ids, the query rows and the slopes of the next piece
// are fetched while the current one is still being consumed.  The cut is computed by every warp from
// context_lens alone (two coalesced passes), so there is no scheduler state in global memory.
//
// When the caller hands over the step's new K/V rows (Algorithm 2, "Store reshaped K, V into C_K, C_V"), the
// worker that is about to fetch the tile holding a sequence's last position stores that sequence's new token
// to its slot first -- plain stores, a generic-to-async proxy fence, then the bulk copy -- so the step needs no
// separate launch for the slot-mapped write.  Every tile belongs to exactly one worker, so nobody else reads
// the row before it is there.
//
// Per tile the warp computes, transposed so that the 16 tokens are the rows and the
// (up to 8) heads of the group the columns of an m16n8k16 tile,
//   S^T = K q^T              8 k-steps over the head dimension          (Eq. 3, dot products)
//   s   = S^T * scale*log2e + slope_h*log2e*(j - (n-1))                 (Eq. 3, ALiBi bias)
//   running max / denominator per head, p = 2^(s - m) rounded to bf16   (Eq. 4, online)
//   O^T += V^T p^T           one m16n8k16 per 16 output dims            (Eq. 5)
// p^T reaches its operand layout through movmatrix; the denominator sums the same
// rounded p that the tensor core multiplies; accumulation is fp32.
#include "tma_mma.cuh"

namespace optgqa {

namespace {

constexpr int kTileTok = 16;                     // tokens per tile (one ring stage holds a K tile and a V tile)
constexpr int kWarps = 4;                        // workers per CTA
constexpr int kStages = 2;                       // ring depth per worker
constexpr int kCtasPerSm = 2;
constexpr int kDescSlots = 4;                    // item descriptors a worker keeps (>= items between prefetch and use)
constexpr unsigned kFull = 0xffffffffu;
constexpr float kMaxSlack = 8.f;                // log2 units by which a score may exceed the running reference maximum

struct StreamParams {
    const __nv_bfloat16* q;
    const int32_t* block_tables;
    const int32_t* context_lens;
    const float* slopes;
    float* partial_out;     // rows of the pieces (see balanced_layout)
    float* partial_lse;
    long long* header;      // {tiles in the stream, workers}
    long long* seq_info;    // per sequence {tiles, partitions} of one head over the earlier sequences
    int* status;
    float scale;
    int B;
    int max_blocks;
    int Hq;
    int Hkv;
    int bs;
    int partition_size;
    int max_partitions;
    int window;             // > 0: only the last `window` keys of each sequence are attended to
    // fused store of the step's new tokens (all null when the cache already holds them)
    const uint4* k_new;
    const uint4* v_new;
    uint4* k_cache_w;
    uint4* v_cache_w;
    const int64_t* slot_mapping;
};

template <int D>
struct StreamCfg {
    static constexpr int NBOX = D / 64;                   // 128-byte-wide boxes per token row
    static constexpr int BOX_BYTES = kTileTok * 128;      // 16 rows x 128 B
    static constexpr int TILE_BYTES = NBOX * BOX_BYTES;   // K (or V) bytes per tile
    static constexpr int WARP_RING = kStages * 2 * TILE_BYTES;
    static constexpr int OFF_DESC = kWarps * WARP_RING;
    static constexpr int OFF_BAR = OFF_DESC + kWarps * kDescSlots * 32;
    static constexpr int SMEM = OFF_BAR + kWarps * kStages * 8 + 1024;   // + slack to align the ring to 1 KB
};

// Transposes an 8x8 matrix of 16-bit elements held one row pair per thread (the ldmatrix layout).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of token row `row` inside a tile stored as
// NBOX boxes of 16 rows x 128 B with the 128-byte swizzle (chunk index XOR row mod 8).
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * (kTileTok * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

__device__ __forceinline__ float group_max(float v) {     // over the 8 lanes that share lane & 3
    v = fmaxf(v, __shfl_xor_sync(kFull, v, 4));
    v = fmaxf(v, __shfl_xor_sync(kFull, v, 8));
    return fmaxf(v, __shfl_xor_sync(kFull, v, 16));
}

__device__ __forceinline__ float group_sum(float v) {
    v += __shfl_xor_sync(kFull, v, 4);
    v += __shfl_xor_sync(kFull, v, 8);
    return v + __shfl_xor_sync(kFull, v, 16);
}

// Position in the tile stream: streams (sequence, KV head) follow one another in that order, each
// ceil(n / 16) tiles long; sequences without tokens take no room.
struct StreamCursor {
    int s, kvh, n;          // sequence, KV head, context length of s
    int tiles, parts;       // tiles and partitions of one stream of s
    int jt;                 // tile inside the stream
    long long pos;          // the same position in the end-to-end numbering
    long long tiles_before; // sum of `tiles` over earlier sequences (one head)
    long long parts_before; // sum of `parts` over earlier sequences (one head)
};

template <int D, int G>
__global__ void __launch_bounds__(kWarps * 32, kCtasPerSm)
decode_stream_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const StreamParams p) {
    using C = StreamCfg<D>;
    constexpr int KS = D / 16;    // k-steps of K q^T
    constexpr int MT = D / 16;    // m-tiles of V^T p^T
    extern __shared__ char smem_raw[];
    char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);

    grid_dependency_launch();   // the grid after this one (the reduce) may start its own prologue
    const uint64_t read_once = l2_policy_evict_first();     // every K/V byte is read exactly once
    const uint64_t keep = l2_policy_evict_last();           // the pieces are read by the merge that follows
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int P = p.partition_size, P16 = P / kTileTok;    // tiles per full partition
    // A sequence's stream starts at the tile that holds its first attended key (tile 0 without a window) and its
    // partitions are counted from there.
    auto first_tile_of = [&](int n) { return p.window > 0 ? max(0, n - p.window) / kTileTok : 0; };
    auto tiles_of = [&](int n) { return (n + kTileTok - 1) / kTileTok - first_tile_of(n); };
    const int* __restrict__ lens = p.context_lens;         // read before the dependency wait: see the ordering contract
    // Entry of a sequence's page table that holds token `tok`.  Held below max_blocks, so that a context length that
    // breaks the caller's promise (n_s <= max_blocks * bs) gives a wrong row and not an access outside the table.
    auto table_index = [&](int tok) { return min(tok / p.bs, p.max_blocks - 1); };   // max_blocks >= 1 (host check)
    if (lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }

    // ------------------------------------------------------------------ this worker's range of the tile stream
    long long total = 0;
    for (int s0 = 0; s0 < p.B; s0 += 32) {
        const int n = s0 + lane < p.B ? __ldg(lens + s0 + lane) : 0;
        int tl = tiles_of(n);
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) tl += __shfl_xor_sync(kFull, tl, o);
        total += tl;
    }
    total *= p.Hkv;
    // Never more workers than tiles, so that every worker's range holds at least one tile.
    const long long grid_workers = (long long)gridDim.x * kWarps, me = (long long)blockIdx.x * kWarps + warp;
    const long long workers = total < grid_workers ? (total > 0 ? total : 1) : grid_workers;
    if (me == 0) {
        grid_dependency_wait();     // the previous reader of the workspace must be done
        if (lane == 0) {
            p.header[0] = total;
            p.header[1] = workers;
        }
    }
    if (total == 0 || me >= workers) return;
    const long long lo = total * me / workers, hi = total * (me + 1) / workers;

    StreamCursor cur;       // the next piece to be described (runs one piece ahead of the issue side)
    {
        // sequence whose tiles contain position lo
        long long acc_t = 0, acc_p = 0;
        cur.s = -1;
        for (int s0 = 0; s0 < p.B && cur.s < 0; s0 += 32) {
            const int n = s0 + lane < p.B ? __ldg(lens + s0 + lane) : 0;
            const int tl = tiles_of(n), np = (tl + P16 - 1) / P16;
            int incl_t = tl, incl_p = np;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int vt = __shfl_up_sync(kFull, incl_t, o), vp = __shfl_up_sync(kFull, incl_p, o);
                if (lane >= o) {
                    incl_t += vt;
                    incl_p += vp;
                }
            }
            const unsigned hit = __ballot_sync(kFull, (acc_t + incl_t) * p.Hkv > lo);
            if (hit) {
                const int src = __ffs(hit) - 1;
                cur.s = s0 + src;
                cur.n = __shfl_sync(kFull, n, src);
                cur.tiles = __shfl_sync(kFull, tl, src);
                cur.parts = __shfl_sync(kFull, np, src);
                cur.tiles_before = acc_t + __shfl_sync(kFull, incl_t, src) - cur.tiles;
                cur.parts_before = acc_p + __shfl_sync(kFull, incl_p, src) - cur.parts;
            } else {
                acc_t += __shfl_sync(kFull, incl_t, 31);
                acc_p += __shfl_sync(kFull, incl_p, 31);
            }
        }
        if (cur.s < 0) return;                               // cannot happen: lo < total
        const int r = (int)(lo - cur.tiles_before * p.Hkv);
        cur.kvh = r / cur.tiles;
        cur.jt = r - cur.kvh * cur.tiles;
        cur.pos = lo;
    }
    auto next_stream = [&]() {
        cur.jt = 0;
        if (++cur.kvh == p.Hkv) {
            cur.kvh = 0;
            cur.tiles_before += cur.tiles;
            cur.parts_before += cur.parts;
            do {
                ++cur.s;
                cur.n = cur.s < p.B ? __ldg(lens + cur.s) : 0;
            } while (cur.s < p.B && cur.n == 0);
            cur.tiles = tiles_of(cur.n);
            cur.parts = (cur.tiles + P16 - 1) / P16;
        }
    };
    auto cur_valid = [&]() { return cur.s < p.B && cur.pos < hi; };
    if (!cur_valid()) return;

    char* ring = smem + warp * C::WARP_RING;
    int4* desc = reinterpret_cast<int4*>(smem + C::OFF_DESC) + warp * (2 * kDescSlots);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR) + warp * kStages;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kStages; ++i) mbar_init(&bars[i], 1);
        fence_barrier_init();
    }
    __syncwarp();

    // Describes the piece under `cur` in slot (piece & 3), starts the loads of its first 32 page ids, moves `cur`
    // on.  A piece is the part of one partition that lies inside this worker's range.  desc[2i] = {s, kvh, n, first tile in the stream}, desc[2i+1] = {tiles, row of the
    // partial result of the group's first head}; tiles are numbered from the sequence's token 0.
    int pieces = 0;               // pieces described so far
    int pages_nxt = 0;            // lane l: physical page of tile l of the piece described last
    auto describe_next = [&]() {
        const int part = cur.jt / P16;
        const int len = (int)min((long long)(min((part + 1) * P16, cur.tiles) - cur.jt), hi - cur.pos);
        // pieces are numbered by (partition index in the end-to-end order) + (worker index): both only grow
        const int obase = (int)((cur.parts_before * p.Hkv + (long long)cur.kvh * cur.parts + part + me) * G);
        if (lane == 0 && cur.kvh == 0 && cur.jt == 0) {
            p.seq_info[2 * cur.s] = cur.tiles_before;
            p.seq_info[2 * cur.s + 1] = cur.parts_before;
        }
        // Where this range and a partition end together inside a stream, the next piece is two numbers on:
        // mark the number in between as empty, so that the merge can sweep the stream's numbers without gaps.
        if (cur.pos + len == hi && cur.jt + len < cur.tiles && (cur.jt + len) % P16 == 0 && lane < G)
            p.partial_lse[obase + G + lane] = -INFINITY;
        if (lane == 0) {
            desc[2 * (pieces & (kDescSlots - 1))] = make_int4(cur.s, cur.kvh, cur.n, first_tile_of(cur.n) + cur.jt);
            desc[2 * (pieces & (kDescSlots - 1)) + 1] = make_int4(len, obase, 0, 0);
        }
        // the piece is streamed from its last tile backwards: page ids of its last block of 32 tiles first
        const int blk = (len - 1) & ~31;
        const int tok = (first_tile_of(cur.n) + cur.jt + blk + lane) * kTileTok;
        pages_nxt = blk + lane < len ? __ldg(p.block_tables + (size_t)cur.s * p.max_blocks + table_index(tok)) : 0;
        ++pieces;
        cur.pos += len;
        cur.jt += len;
        if (cur.jt == cur.tiles) next_stream();
        __syncwarp();
    };

    // ------------------------------------------------------------------ issue side
    int is_piece = -1, is_j = 0, is_ntile = 0, is_kvh = 0, is_tile0 = 0, is_s = 0, is_last_tile = -1;
    int pages_cur = 0;
    uint32_t issued = 0, consumed = 0;     // tiles over the worker's whole stream: ring slot = count % kStages
    int cs_piece = -1;
    // B fragments of q for the piece entered last on the issue side (rows = heads; heads >= G are zero), its slopes
    uint32_t q_nxt[KS][2];
    float sl_nxt[2];
    const float qscale = p.scale * kLog2e;

    auto issue_one = [&]() {               // precondition: a tile may be issued
        if (is_j == is_ntile) {
            // enter the next piece: its descriptor and first page ids were produced one piece ago
            ++is_piece;
            const int4 d0 = desc[2 * (is_piece & (kDescSlots - 1))];
            is_ntile = desc[2 * (is_piece & (kDescSlots - 1)) + 1].x;
            pages_cur = pages_nxt;
            is_j = 0;
            is_s = d0.x;
            is_kvh = d0.y;
            is_tile0 = d0.w;
            is_last_tile = (d0.z - 1) / kTileTok;          // the tile that holds the sequence's newest token
            // q may be the output of the kernel that precedes this one in the stream (the Q/K/V projection, which
            // lets its dependents start early): it is read only after the dependency wait, and from L2, never through
            // a non-coherent path that could hold a line fetched before that kernel's stores.
            const uint32_t* qh = reinterpret_cast<const uint32_t*>(
                p.q + ((size_t)d0.x * p.Hq + (size_t)d0.y * G + (g < G ? g : 0)) * D);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                q_nxt[ks][0] = g < G ? __ldcg(qh + ks * 8 + t) : 0u;
                q_nxt[ks][1] = g < G ? __ldcg(qh + ks * 8 + 4 + t) : 0u;
            }
#pragma unroll
            for (int c = 0; c < 2; ++c)
                sl_nxt[c] = (p.slopes && 2 * t + c < G) ? __ldg(p.slopes + d0.y * G + 2 * t + c) * kLog2e : 0.f;
            if (cur_valid()) describe_next();
        } else if (((is_ntile - 1 - is_j) & 31) == 31) {
            // pieces longer than 512 tokens: the page ids of the block of 32 tiles below
            const int tok = (is_tile0 + (is_ntile - 32 - is_j) + lane) * kTileTok;
            pages_cur = __ldg(p.block_tables + (size_t)is_s * p.max_blocks + table_index(tok));
        }
        const int is_r = is_ntile - 1 - is_j;      // tile inside the piece: from the last one backwards
        if (p.k_new && is_tile0 + is_r == is_last_tile) {
            // The step's new token of this sequence lies in the tile about to be fetched: store its K and V rows
            // of this head first (as the slot-mapped write would), and order the stores before the bulk copy.
            const long long slot = __ldg(p.slot_mapping + is_s);
            if (slot >= 0) {
                constexpr int VEC = D * 2 / 16;                  // 16-byte vectors per row
                if (lane < 2 * VEC) {
                    const bool is_v = lane >= VEC;
                    const int vi = lane % VEC;
                    const size_t src = ((size_t)is_s * p.Hkv + is_kvh) * VEC + vi;
                    const size_t dst = (((size_t)(slot / p.bs) * p.Hkv + is_kvh) * p.bs + (size_t)(slot % p.bs)) * VEC + vi;
                    if (is_v) p.v_cache_w[dst] = __ldg(p.v_new + src);
                    else p.k_cache_w[dst] = __ldg(p.k_new + src);
                }
                asm volatile("fence.proxy.async.global;" ::: "memory");
            }
            __syncwarp();
        }
        const int phys = __shfl_sync(kFull, pages_cur, is_r & 31);
        if (lane == 0) {
            const int tok = (is_tile0 + is_r) * kTileTok;
            const int row = (phys * p.Hkv + is_kvh) * p.bs + tok % p.bs;       // row of the [rows, D] view
            const int st = issued % kStages;
            char* dst = ring + st * 2 * C::TILE_BYTES;
            mbar_expect_tx(&bars[st], 2 * C::TILE_BYTES);
#pragma unroll
            for (int b = 0; b < C::NBOX; ++b) {
                tma_load_2d_hint(dst + b * C::BOX_BYTES, &map_k, b * 64, row, &bars[st], read_once);
                tma_load_2d_hint(dst + C::TILE_BYTES + b * C::BOX_BYTES, &map_v, b * 64, row, &bars[st], read_once);
            }
        }
        ++is_j;
        ++issued;
    };
    // A tile may be issued while a ring slot is free and there is a tile left; a new piece is entered only
    // once the consume side has entered the one before it (q_nxt / sl_nxt hold one piece).
    auto issue_allowed = [&]() {
        if (issued - consumed >= (uint32_t)kStages) return false;
        if (is_j < is_ntile) return true;
        return is_piece < pieces - 1 && is_piece <= cs_piece;
    };

    {
        // While the preceding grid drains: bring the first piece's page ids towards this SM (the page table is
        // complete before the call, see the ordering contract in the header), and ask L2 -- the point of coherence,
        // where a line can never be stale -- for the query rows, which the preceding grid may still be writing.
        const int part = cur.jt / P16;
        const int len = (int)min((long long)(min((part + 1) * P16, cur.tiles) - cur.jt), hi - cur.pos);
        const int blk = (len - 1) & ~31;
        const int tok = (first_tile_of(cur.n) + cur.jt + blk + lane) * kTileTok;
        if (blk + lane < len)
            asm volatile("prefetch.global.L1 [%0];" ::"l"(p.block_tables + (size_t)cur.s * p.max_blocks + table_index(tok)));
        if (lane < G * D * 2 / 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(
                reinterpret_cast<const char*>(p.q + ((size_t)cur.s * p.Hq + (size_t)cur.kvh * G) * D) + lane * 128));
    }
    grid_dependency_wait();     // the cache may still be receiving this step's appended tokens
    describe_next();            // piece 0
    while (issue_allowed()) issue_one();

    // ------------------------------------------------------------------ consume side
    uint32_t qb[KS][2];
    float sl[2] = {0.f, 0.f};
    float o[MT][4];
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    int cs_j = 0, cs_ntile = 0, cs_n = 0, cs_tile0 = 0, cs_obase = 0;
    const int lrow = lane & 7, lmat = lane >> 3;
    bool ok = true;

    while (consumed != issued) {
        if (cs_j == cs_ntile) {
            // enter the next piece
            ++cs_piece;
            const int4 d0 = desc[2 * (cs_piece & (kDescSlots - 1))], d1 = desc[2 * (cs_piece & (kDescSlots - 1)) + 1];
            cs_n = d0.z;
            cs_tile0 = d0.w;
            cs_ntile = d1.x;
            cs_obase = d1.y;
            cs_j = 0;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qb[ks][0] = q_nxt[ks][0];
                qb[ks][1] = q_nxt[ks][1];
            }
            sl[0] = sl_nxt[0];
            sl[1] = sl_nxt[1];
#pragma unroll
            for (int i = 0; i < MT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
            m0 = m1 = -INFINITY;
            l0 = l1 = 0.f;
        }
        const int st = consumed % kStages;
        char* kst = ring + st * 2 * C::TILE_BYTES;
        char* vst = kst + C::TILE_BYTES;
        ok = __all_sync(kFull, mbar_wait(&bars[st], (consumed / kStages) & 1, p.status));
        if (!ok) break;

        const int j0 = (cs_tile0 + (cs_ntile - 1 - cs_j)) * kTileTok;
        const int valid = min(kTileTok, cs_n - j0);
        if (valid < kTileTok) {
            // Rows past the end of the sequence hold whatever the page held: zero the V rows so that
            // 0 * garbage cannot produce NaN (their scores are masked below).
            for (int r = valid + (lane >> 3); r < kTileTok; r += 4)
#pragma unroll
                for (int b = 0; b < C::NBOX; ++b)
                    *reinterpret_cast<uint4*>(vst + b * C::BOX_BYTES + r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
            __syncwarp();
        }

        // ---- S^T[token][head]: rows = the tile's 16 tokens, columns = heads of the group
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
        {
            // two accumulators, so that the k-steps form two dependency chains of half the length
            float sd[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t kbase = smem_u32(kst);
            const int krow = lrow + 8 * (lmat & 1);          // matrices 0,2: tokens 0-7; 1,3: tokens 8-15
#pragma unroll
            for (int ks = 0; ks < KS; ks += 2) {
                uint32_t a[4], b[4];
                ldmatrix_x4(a, kbase + swz(krow, 2 * ks + (lmat >> 1)));
                ldmatrix_x4(b, kbase + swz(krow, 2 * ks + 2 + (lmat >> 1)));
                mma_bf16(sc, a, qb[ks][0], qb[ks][1]);
                mma_bf16(sd, b, qb[ks + 1][0], qb[ks + 1][1]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) sc[i] += sd[i];
        }
        // thread holds tokens j0 + g (sc[0], sc[1]) and j0 + g + 8 (sc[2], sc[3]) for heads 2t, 2t + 1
        {
            const int ja = j0 + g;
            const float relA = (float)(ja - (cs_n - 1)), relB = relA + 8.f;
            sc[0] = fmaf(sc[0], qscale, sl[0] * relA);
            sc[1] = fmaf(sc[1], qscale, sl[1] * relA);
            sc[2] = fmaf(sc[2], qscale, sl[0] * relB);
            sc[3] = fmaf(sc[3], qscale, sl[1] * relB);
            const int cs_start = p.window > 0 ? max(0, cs_n - p.window) : 0;     // first attended key
            if (ja >= cs_n || ja < cs_start) sc[0] = sc[1] = -INFINITY;
            if (ja + 8 >= cs_n || ja + 8 < cs_start) sc[2] = sc[3] = -INFINITY;
        }
        // Running maximum per head, kept lazily: the tiles of a piece come from its last one backwards, so the ALiBi
        // term only falls after the first tile and the reference m rarely has to move.  It moves (and the
        // accumulators are rescaled) only when some score exceeds it by more than kMaxSlack; until then p may be
        // as large as 2^kMaxSlack, which bf16 and the fp32 sums hold as well as values below 1.
        const float x0 = fmaxf(sc[0], sc[2]), x1 = fmaxf(sc[1], sc[3]);
        if (__any_sync(kFull, x0 > m0 + kMaxSlack || x1 > m1 + kMaxSlack)) {
            const float m0n = fmaxf(m0, group_max(x0)), m1n = fmaxf(m1, group_max(x1));
            const float a0 = ex2(m0 - m0n), a1 = ex2(m1 - m1n);
            m0 = m0n;
            m1 = m1n;
            l0 *= a0;
            l1 *= a1;
#pragma unroll
            for (int i = 0; i < MT; ++i) {
                o[i][0] *= a0;
                o[i][1] *= a1;
                o[i][2] *= a0;
                o[i][3] *= a1;
            }
        }
        // p rounded to bf16 once: the same values feed the tensor core and the denominator
        const __nv_bfloat162 pa = __floats2bfloat162_rn(ex2(sc[0] - m0), ex2(sc[1] - m1));   // token g
        const __nv_bfloat162 pb = __floats2bfloat162_rn(ex2(sc[2] - m0), ex2(sc[3] - m1));   // token g + 8
        const float2 fa = __bfloat1622float2(pa), fb = __bfloat1622float2(pb);
        l0 += fa.x + fb.x;
        l1 += fa.y + fb.y;
        const uint32_t b0 = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&pa));   // tokens 2t, 2t+1 of head g
        const uint32_t b1 = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&pb));   // tokens 2t+8, 2t+9

        // ---- O^T[dim][head] += V^T[dim][token] * p^T[token][head]; V transposed on the fly by ldmatrix.trans
        {
            const uint32_t vbase = smem_u32(vst);
            const int vrow = lrow + 8 * (lmat >> 1);         // matrices 0,1: tokens 0-7; 2,3: tokens 8-15
#pragma unroll
            for (int i = 0; i < MT; ++i) {
                uint32_t a[4];
                ldmatrix_x4_trans(a, vbase + swz(vrow, 2 * i + (lmat & 1)));
                mma_bf16(o[i], a, b0, b1);
            }
        }
        ++cs_j;
        ++consumed;

        if (cs_j == cs_ntile) {
            // ---- the piece is complete: normalise, write the partial result and its log-sum-exp
            const float L0 = group_sum(l0), L1 = group_sum(l1);
            const float i0 = 1.f / L0, i1 = 1.f / L1;
            if (2 * t < G) {
                const size_t row = (size_t)cs_obase + (size_t)(2 * t);
                float* po = p.partial_out + row * D;
#pragma unroll
                for (int i = 0; i < MT; ++i) {
                    st_global_hint(po + 16 * i + g, o[i][0] * i0, keep);
                    st_global_hint(po + 16 * i + 8 + g, o[i][2] * i0, keep);
                }
                if (g == 0) st_global_hint(p.partial_lse + row, (m0 + lg2(L0)) * kLn2, keep);
            }
            if (2 * t + 1 < G) {
                const size_t row = (size_t)cs_obase + (size_t)(2 * t + 1);
                float* po = p.partial_out + row * D;
#pragma unroll
                for (int i = 0; i < MT; ++i) {
                    st_global_hint(po + 16 * i + g, o[i][1] * i1, keep);
                    st_global_hint(po + 16 * i + 8 + g, o[i][3] * i1, keep);
                }
                if (g == 0) st_global_hint(p.partial_lse + row, (m1 + lg2(L1)) * kLn2, keep);
            }
        }

        // Where this warp wrote into the slot just consumed (the zeroed rows), order those generic-proxy writes
        // before the async-proxy copy that refills it.  Reads need no fence: the fragments are in registers by the
        // time the instructions that use them have been issued.
        if (valid < kTileTok) fence_proxy_async();
        __syncwarp();
        while (issue_allowed()) issue_one();
    }

    if (!ok) {
        // A wait gave up (already recorded).  Give the copies still in flight one more bounded
        // chance to land before this CTA's shared memory is released.
        for (uint32_t kk = consumed; kk != issued; ++kk) mbar_wait(&bars[kk % kStages], (kk / kStages) & 1, p.status);
    }
}

// One resident wave; never more workers than there could be 16-token tiles (the ranges are cut at tile granularity),
// nor than the workspace has room for.  A grid that leaves some SMs with one CTA and others with two would undo the
// balance.
long long stream_grid_ctas(int B, int Hkv, int max_partitions, int partition_size) {
    const int sms = sm_count();
    if (sms <= 0) return 0;
    const long long items = (long long)B * Hkv * max_partitions * (partition_size / kTileTok);
    long long ctas = (items + kWarps - 1) / kWarps;
    if (ctas > (long long)sms * kCtasPerSm) ctas = (long long)sms * kCtasPerSm;
    if (ctas > kBalancedMaxWorkers / kWarps) ctas = kBalancedMaxWorkers / kWarps;
    return ctas;
}

template <int D, int G>
int launch_one(const CUtensorMap& mk, const CUtensorMap& mv, const StreamParams& p, cudaStream_t stream) {
    using C = StreamCfg<D>;
    static std::atomic<bool> configured[kMaxDevices];
    if (!ensure_smem_limit(decode_stream_kernel<D, G>, C::SMEM, configured)) return OPT_GQA_ERR_CUDA;
    const long long ctas = stream_grid_ctas(p.B, p.Hkv, p.max_partitions, p.partition_size);
    if (ctas <= 0) return OPT_GQA_ERR_CUDA;
    return launch_dependent(decode_stream_kernel<D, G>, dim3((unsigned)ctas), dim3(kWarps * 32), C::SMEM, stream, mk,
                            mv, p);
}

template <int D>
int launch_g(const CUtensorMap& mk, const CUtensorMap& mv, const StreamParams& p, int G, cudaStream_t stream) {
    switch (G) {
        case 1: return launch_one<D, 1>(mk, mv, p, stream);
        case 2: return launch_one<D, 2>(mk, mv, p, stream);
        case 4: return launch_one<D, 4>(mk, mv, p, stream);
        case 8: return launch_one<D, 8>(mk, mv, p, stream);
    }
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace

int sm_count() {
    static std::atomic<int> counts[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    int c = counts[dev].load(std::memory_order_relaxed);
    if (!c) {
        if (cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        counts[dev].store(c, std::memory_order_relaxed);
    }
    return c;
}

long long stream_grid_workers(int B, int Hkv, int max_partitions, int partition_size) {
    return stream_grid_ctas(B, Hkv, max_partitions, partition_size) * kWarps;
}

// Pieces and bookkeeping go to `workspace` (see balanced_layout).  One partial per whole partition is the tile
// kernel's job (decode_tc.cu, one CTA per partition).
int launch_decode_stream(const void* q, const void* k_cache, const void* v_cache, const int32_t* block_tables,
                         int max_blocks_per_seq, const int32_t* context_lens, const float* alibi_slopes, float scale,
                         int B, int Hq, int Hkv, int D, int bs, int64_t num_blocks, int partition_size,
                         void* workspace, int max_partitions, int window, int* device_status, cudaStream_t stream,
                         const FusedAppend* append) {
    if (!workspace) return OPT_GQA_ERR_NULL;
    const uint64_t rows = (uint64_t)num_blocks * (uint64_t)Hkv * (uint64_t)bs;
    if (rows == 0 || rows > 0x7fffffffull) return OPT_GQA_ERR_SHAPE;
    CUtensorMap mk, mv;
    if (!make_cache_map(&mk, k_cache, rows, D, kTileTok) || !make_cache_map(&mv, v_cache, rows, D, kTileTok))
        return OPT_GQA_ERR_CUDA;
    const BalancedLayout L = balanced_layout(B, Hq, Hkv, D, max_partitions);
    if (L.rows > 0x7fffffffull) return OPT_GQA_ERR_SHAPE;
    char* ws = static_cast<char*>(workspace);
    StreamParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.block_tables = block_tables;
    p.context_lens = context_lens;
    p.slopes = alibi_slopes;
    p.header = reinterpret_cast<long long*>(ws + L.header);
    p.seq_info = reinterpret_cast<long long*>(ws + L.seq_info);
    p.partial_lse = reinterpret_cast<float*>(ws + L.lse);
    p.partial_out = reinterpret_cast<float*>(ws + L.out);
    p.status = device_status;
    p.scale = scale;
    p.B = B;
    p.max_blocks = max_blocks_per_seq;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.bs = bs;
    p.partition_size = partition_size;
    p.max_partitions = max_partitions;
    p.window = window;
    p.k_new = append ? static_cast<const uint4*>(append->k_new) : nullptr;
    p.v_new = append ? static_cast<const uint4*>(append->v_new) : nullptr;
    p.k_cache_w = append ? static_cast<uint4*>(append->k_cache) : nullptr;
    p.v_cache_w = append ? static_cast<uint4*>(append->v_cache) : nullptr;
    p.slot_mapping = append ? append->slot_mapping : nullptr;
    const int G = Hq / Hkv;
    if (D == 128) return launch_g<128>(mk, mv, p, G, stream);
    if (D == 64) return launch_g<64>(mk, mv, p, G, stream);
    return OPT_GQA_ERR_SHAPE;
}

}  // namespace optgqa

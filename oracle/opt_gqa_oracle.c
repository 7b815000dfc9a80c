/*
 * Opt-GQA CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 statement of what the Opt-GQA attention path computes:
 * grouped-query attention over a paged key/value cache with an ALiBi linear
 * bias.  It exists so the CUDA library can be checked against something that
 * can be verified against the paper by eye.  It shares no source, header,
 * table or helper with the CUDA path; only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.
 *
 * Everything here is the definition written out: no blocking, no fusion, no
 * online softmax, no reordering.  Inputs are the exact fp32 / bf16 values the
 * GPU sees, widened to double (exact); all arithmetic is double.
 *
 * Array layouts (row-major, last index fastest):
 *   q              [T, Hq, D]                  T = number of query tokens
 *   k_cache/v_cache[num_blocks, Hkv, bs, D]    the paged pool
 *   block_tables   [B, max_blocks]  int32      logical page i of seq s -> physical page
 *   context_lens   [B]              int32      tokens of seq s in the cache (incl. new ones)
 *   q_start_loc    [B+1]            int32      prefix sums of new-token counts (NULL: one per seq)
 *   out            [T, Hq, D]       double
 * dtype: 0 = fp32 storage, 1 = bf16 storage (uint16 bit patterns).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* exact widening of one stored element to double */
static double load_elem(const void* base, int64_t idx, int dtype) {
    if (dtype == 0) {
        return (double)((const float*)base)[idx];
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16; /* bf16 = top half of fp32 */
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/*
 * ALiBi slopes for a power-of-two head count: slope_h = 2^(-8 (h+1) / Hq),
 * h = 0..Hq-1 (the geometric sequence of the ALiBi construction the paper's
 * "Integration and Optimization of ALiBi" paragraph refers to; Algorithm 1,
 * "Create ALiBi bias").
 */
void oracle_alibi_slopes(int Hq, double* slopes) {
    for (int h = 0; h < Hq; ++h) slopes[h] = pow(2.0, -8.0 * (double)(h + 1) / (double)Hq);
}

/*
 * Algorithm 1, "Reshape and store K, V into C_K, C_V" (also Algorithm 2, and
 * Eq. 2: the cached sequence is the previous tokens followed by the new ones).
 * Token t of the new K/V goes to slot = slot_mapping[t]: page slot / bs,
 * offset slot % bs.  Negative slot: the token is skipped.  Pure byte copy.
 * Returns 0, or -1 if a slot lies outside the pool.
 */
int oracle_cache_append(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                        const int64_t* slot_mapping, int T, int Hkv, int D, int bs,
                        int64_t num_blocks, int dtype) {
    const size_t es = dtype == 0 ? 4 : 2;
    const size_t row = (size_t)D * es;
    for (int t = 0; t < T; ++t) {
        int64_t slot = slot_mapping[t];
        if (slot < 0) continue;
        int64_t page = slot / bs, off = slot % bs;
        if (page >= num_blocks) return -1;
        for (int h = 0; h < Hkv; ++h) {
            size_t src = ((size_t)t * Hkv + h) * row;
            size_t dst = ((((size_t)page * Hkv + h) * bs) + off) * row;
            memcpy((char*)k_cache + dst, (const char*)k_new + src, row);
            memcpy((char*)v_cache + dst, (const char*)v_new + src, row);
        }
    }
    return 0;
}

/*
 * Attention of ONE query row against logical keys j in [j_lo, j_hi) of its
 * sequence, Eq. 3 -> Eq. 4 -> Eq. 5:
 *   raw_j = scale * <q, k_j> + bias_j ,  bias_j = -slope * (pos - j)      (Eq. 3)
 *   w_j   = exp(raw_j) / sum_j' exp(raw_j')                               (Eq. 4)
 *   o     = sum_j w_j v_j                                                 (Eq. 5)
 * The dot product is scaled, the bias is not (the text after Eq. 2 scales the
 * dot product first and adds the mask afterwards).  The maximum is subtracted
 * before exp, which leaves Eq. 4 unchanged.  Also returns
 * lse = log sum_j exp(raw_j)  (-inf for an empty range, o = 0 then).
 * k_j / v_j are found through the block table: logical token j lives in page
 * table[j / bs] at offset j % bs, head kvh ("Shared Key-Value": the G query
 * heads of a group read the same K/V head).
 */
static void attend_row(double* o, double* lse_out, const void* q, int64_t q_off, const void* k_cache,
                       const void* v_cache, const int32_t* table, int kvh, int Hkv, int D, int bs,
                       int dtype, double scale, double slope, int64_t pos, int64_t j_lo, int64_t j_hi) {
    int64_t n = j_hi - j_lo;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (n <= 0) {
        *lse_out = -INFINITY;
        return;
    }
    double* raw = (double*)malloc(sizeof(double) * (size_t)n);
    double mx = -INFINITY;
    for (int64_t j = j_lo; j < j_hi; ++j) {
        int64_t page = table[j / bs], off = j % bs;
        int64_t base = (((page * Hkv + kvh) * bs) + off) * (int64_t)D;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += load_elem(q, q_off + d, dtype) * load_elem(k_cache, base + d, dtype);
        double r = scale * dot - slope * (double)(pos - j);
        raw[j - j_lo] = r;
        if (r > mx) mx = r;
    }
    double denom = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        raw[i] = exp(raw[i] - mx);
        denom += raw[i];
    }
    for (int64_t j = j_lo; j < j_hi; ++j) {
        int64_t page = table[j / bs], off = j % bs;
        int64_t base = (((page * Hkv + kvh) * bs) + off) * (int64_t)D;
        double w = raw[j - j_lo] / denom;
        for (int d = 0; d < D; ++d) o[d] += w * load_elem(v_cache, base + d, dtype);
    }
    *lse_out = mx + log(denom);
    free(raw);
}

/*
 * Algorithm 2, "Compute context attention with caches" (decode: q_start_loc
 * NULL, one query token per sequence at position n-1) and the prompt branch
 * over the paged cache (q_start_loc given: new token i of sequence s sits at
 * position pos = n_s - q_len_s + i and sees keys j <= pos, "causal mask +
 * ALiBi bias").  Query head h uses K/V head h / G, G = Hq / Hkv (consecutive
 * heads form a group).  slopes may be NULL (all zero).  A sequence with
 * n_s = 0 gives zero rows.  window > 0 additionally restricts keys to
 * pos - j < window (Algorithm 1's "local" mask); 0 = no window.
 */
int oracle_paged_attention(double* out, const void* q, const void* k_cache, const void* v_cache,
                           const int32_t* block_tables, int max_blocks, const int32_t* context_lens,
                           const int32_t* q_start_loc, const double* slopes, double scale, int B, int Hq,
                           int Hkv, int D, int bs, int dtype, int window) {
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < B; ++s) {
        for (int h = 0; h < Hq; ++h) {
            const int64_t n = context_lens[s];
            const int64_t t0 = q_start_loc ? q_start_loc[s] : s;
            const int64_t qlen = q_start_loc ? (q_start_loc[s + 1] - q_start_loc[s]) : 1;
            const double slope = slopes ? slopes[h] : 0.0;
            for (int64_t i = 0; i < qlen; ++i) {
                const int64_t pos = n - qlen + i;
                int64_t j_lo = 0, j_hi = pos + 1;
                if (window > 0 && pos + 1 - window > 0) j_lo = pos + 1 - window;
                if (j_hi < 0) j_hi = 0;
                double lse;
                attend_row(out + ((t0 + i) * Hq + h) * D, &lse, q, ((t0 + i) * Hq + h) * (int64_t)D, k_cache,
                           v_cache, block_tables + (int64_t)s * max_blocks, h / G, Hkv, D, bs, dtype, scale,
                           slope, pos, j_lo, j_hi);
            }
        }
    }
    return 0;
}

/*
 * Long-sequence partitioning (the paragraph before Eq. 1: the context is cut
 * into partitions of P tokens and attention is computed separately for each).
 * For decode, partition p of sequence s covers keys [pP, min((p+1)P, n_s)).
 * Outputs the per-partition normalised result o_p and lse_p (-inf and zeros
 * for partitions beyond the sequence's length).
 *   partial_out [B, Hq, max_partitions, D], partial_lse [B, Hq, max_partitions]
 */
int oracle_partition_partials(double* partial_out, double* partial_lse, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* block_tables, int max_blocks,
                              const int32_t* context_lens, const double* slopes, double scale, int B, int Hq,
                              int Hkv, int D, int bs, int dtype, int P, int max_partitions) {
    if (Hkv <= 0 || Hq % Hkv != 0 || P <= 0) return -1;
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < B; ++s) {
        for (int h = 0; h < Hq; ++h) {
            const int64_t n = context_lens[s];
            const double slope = slopes ? slopes[h] : 0.0;
            for (int p = 0; p < max_partitions; ++p) {
                int64_t j_lo = (int64_t)p * P, j_hi = j_lo + P;
                if (j_hi > n) j_hi = n;
                int64_t row = ((int64_t)s * Hq + h) * max_partitions + p;
                attend_row(partial_out + row * D, partial_lse + row, q, ((int64_t)s * Hq + h) * D, k_cache,
                           v_cache, block_tables + (int64_t)s * max_blocks, h / G, Hkv, D, bs, dtype, scale,
                           slope, n - 1, j_lo, j_hi);
            }
        }
    }
    return 0;
}

/*
 * Combining the partitions (the paragraph before Eq. 1 keeps each partition's
 * output and feeds it into the sequence's result): softmax over the whole
 * context splits exactly as
 *   out = sum_p e^{lse_p} o_p / sum_p e^{lse_p},  p < ceil(n_s / P),
 * evaluated with the largest lse subtracted.  n_s = 0 gives zeros.
 */
int oracle_reduce(double* out, const double* partial_out, const double* partial_lse,
                  const int32_t* context_lens, int B, int Hq, int D, int P, int max_partitions) {
    if (P <= 0) return -1;
    for (int s = 0; s < B; ++s) {
        int64_t n = context_lens[s];
        int np = (int)((n + P - 1) / P);
        if (np > max_partitions) return -1;
        for (int h = 0; h < Hq; ++h) {
            int64_t row0 = ((int64_t)s * Hq + h) * max_partitions;
            double* o = out + ((int64_t)s * Hq + h) * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            double L = -INFINITY;
            for (int p = 0; p < np; ++p)
                if (partial_lse[row0 + p] > L) L = partial_lse[row0 + p];
            if (np == 0 || L == -INFINITY) continue;
            double denom = 0.0;
            for (int p = 0; p < np; ++p) denom += exp(partial_lse[row0 + p] - L);
            for (int p = 0; p < np; ++p) {
                double w = exp(partial_lse[row0 + p] - L) / denom;
                for (int d = 0; d < D; ++d) o[d] += w * partial_out[(row0 + p) * D + d];
            }
        }
    }
    return 0;
}

/*
 * Gather one sequence's K or V head into logical order (Eq. 2: concatenation
 * of the cached blocks along the token axis): dst [n, D] double.
 */
void oracle_unpage(double* dst, const void* cache, const int32_t* table, int n, int kvh, int Hkv, int D,
                   int bs, int dtype) {
    for (int64_t j = 0; j < n; ++j) {
        int64_t page = table[j / bs], off = j % bs;
        int64_t base = (((page * Hkv + kvh) * bs) + off) * (int64_t)D;
        for (int d = 0; d < D; ++d) dst[j * D + d] = load_elem(cache, base + d, dtype);
    }
}

/*
 * The prompt branch with empty caches (Algorithm 1: "Caches are empty" -> GQA grouping -> "Create ALiBi
 * bias" / causal mask -> scores, softmax, weighted sum; Eq. 3-5).  q [T, Hq, D], k, v [T, Hkv, D] are
 * contiguous; sequence s owns rows q_start_loc[s] .. q_start_loc[s+1]-1 and token i of it sees keys
 * 0 .. i of the same sequence:
 *   raw_j = scale * <q_i, k_j> - slope_h * (i - j),  w = softmax_j(raw),  out_i = sum_j w_j v_j.
 * Query head h uses K/V head h / G.
 */
int oracle_prompt_attention(double* out, const void* q, const void* k, const void* v, const int32_t* q_start_loc,
                            const double* slopes, double scale, int B, int Hq, int Hkv, int D, int dtype) {
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int s = 0; s < B; ++s) {
        for (int h = 0; h < Hq; ++h) {
            const int64_t t0 = q_start_loc[s], len = q_start_loc[s + 1] - q_start_loc[s];
            const double slope = slopes ? slopes[h] : 0.0;
            double* raw = (double*)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
            for (int64_t i = 0; i < len; ++i) {
                const int64_t qo = ((t0 + i) * Hq + h) * (int64_t)D;
                double mx = -INFINITY;
                for (int64_t j = 0; j <= i; ++j) {
                    const int64_t ko = ((t0 + j) * Hkv + h / G) * (int64_t)D;
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += load_elem(q, qo + d, dtype) * load_elem(k, ko + d, dtype);
                    raw[j] = scale * dot - slope * (double)(i - j);
                    if (raw[j] > mx) mx = raw[j];
                }
                double denom = 0.0;
                for (int64_t j = 0; j <= i; ++j) {
                    raw[j] = exp(raw[j] - mx);
                    denom += raw[j];
                }
                double* o = out + qo;
                for (int d = 0; d < D; ++d) o[d] = 0.0;
                for (int64_t j = 0; j <= i; ++j) {
                    const int64_t vo = ((t0 + j) * Hkv + h / G) * (int64_t)D;
                    const double w = raw[j] / denom;
                    for (int d = 0; d < D; ++d) o[d] += w * load_elem(v, vo + d, dtype);
                }
            }
            free(raw);
        }
    }
    return 0;
}

/*
 * Q/K/V projection of Eq. 1 (Q = X W_Q, K = X W_K, V = X W_V) with the three weight matrices stored
 * side by side as one 4-bit group-quantised matrix W [K, N], N = (Hq + 2 Hkv) D.  The paper names GPTQ
 * in its title but states no storage format; the reading taken here is the common group-wise one:
 *
 *   qweight [K/8, N]   uint32   code of row 8r+i, column n in bits 4i..4i+3 of word (r, n)
 *   scales  [K/gs, N]  bf16     one scale per group of gs consecutive rows and column
 *   qzeros  [K/gs, N/8] uint32  zero point of group g, column 8c+i in bits 4i..4i+3 of word (g, c)
 *   w[k][n] = scales[k/gs][n] * (code[k][n] - zero[k/gs][n])
 *   y[t][n] = sum_k x[t][k] * w[k][n]        x [T, K] bf16, y [T, N] double
 *
 * Columns 0 .. Hq D - 1 of y are the token's query, the next Hkv D its key, the last Hkv D its value.
 */
int oracle_qkv_project_int4(double* y, const void* x, const uint32_t* qweight, const void* scales,
                            const uint32_t* qzeros, int T, int K, int N, int gs) {
    if (T < 0 || K <= 0 || N <= 0 || gs <= 0 || K % 8 != 0 || N % 8 != 0 || K % gs != 0) return -1;
    #pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                int g = k / gs;
                int code = (int)((qweight[(int64_t)(k / 8) * N + n] >> (4 * (k % 8))) & 0xFu);
                int zero = (int)((qzeros[(int64_t)g * (N / 8) + n / 8] >> (4 * (n % 8))) & 0xFu);
                double w = load_elem(scales, (int64_t)g * N + n, 1) * (double)(code - zero);
                acc += load_elem(x, (int64_t)t * K + k, 1) * w;
            }
            y[(int64_t)t * N + n] = acc;
        }
    }
    return 0;
}

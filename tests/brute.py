"""A second, independent statement of the attention definition, in dense numpy.

Used only to pin the C oracle on tiny inputs: the paged pool is un-paged with
numpy indexing, the full score matrix is materialised, and softmax(scale*QK^T +
bias) V is evaluated with matrix products.  Shares nothing with the oracle or
the CUDA path.
"""
import numpy as np


def widen(a: np.ndarray) -> np.ndarray:
    """fp32 array or uint16 bf16 bit patterns -> float64."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def logical_kv(cache: np.ndarray, table: np.ndarray, n: int) -> np.ndarray:
    """[num_blocks, Hkv, bs, D] + table -> [Hkv, n, D] in token order."""
    bs = cache.shape[2]
    npages = (n + bs - 1) // bs
    pages = widen(cache[table[:npages]])                 # [npages, Hkv, bs, D]
    seq = pages.transpose(1, 0, 2, 3).reshape(cache.shape[1], npages * bs, cache.shape[3])
    return seq[:, :n]


def dense_attention(q, k_cache, v_cache, block_tables, context_lens, slopes, scale, q_start_loc=None, window=0):
    """float64 [T, Hq, D]; decode when q_start_loc is None."""
    T, Hq, D = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    out = np.zeros((T, Hq, D))
    qd = widen(q)
    for s in range(block_tables.shape[0]):
        n = int(context_lens[s])
        if q_start_loc is None:
            rows = np.array([s])
        else:
            rows = np.arange(q_start_loc[s], q_start_loc[s + 1])
        if n == 0 or rows.size == 0:
            continue
        K = logical_kv(k_cache, block_tables[s], n)
        V = logical_kv(v_cache, block_tables[s], n)
        pos = n - rows.size + np.arange(rows.size)       # query positions
        j = np.arange(n)
        rel = pos[:, None] - j[None, :]                  # query_pos - key_pos
        for h in range(Hq):
            S = scale * (qd[rows, h] @ K[h // G].T)
            sl = 0.0 if slopes is None else float(slopes[h])
            S = S - sl * rel
            S = np.where(rel < 0, -np.inf, S)
            if window > 0:
                S = np.where(rel >= window, -np.inf, S)
            S = S - S.max(axis=1, keepdims=True)
            W = np.exp(S)
            W /= W.sum(axis=1, keepdims=True)
            out[rows, h] = W @ V[h // G]
    return out

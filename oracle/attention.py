"""Oracle: grouped-query decode attention, dense and paged (fp64).

TEST INFRASTRUCTURE ONLY - never imported by the product path.

The paper does not define an attention variant of its own: decoding is the
stock transformer decode step whose time Sec. 2 ("Latency Bottleneck",
Fig. 2c) and Table 3 attribute to "decoding".  What is computed here is the
textbook definition for one new token per trace:

    o_h = sum_j softmax_j( q_h . k_j / sqrt(d) ) v_j ,   j in [0, S_t)

with query head h reading KV head h // G (G = Hq / Hkv, consecutive query
heads share a KV head).  The query attends to every stored position including
its own; there is no mask.  S_t = 0 yields zeros.

All arithmetic is float64.  Inputs that were stored in a narrower type are
upcast exactly by the caller before they get here.
"""
from __future__ import annotations

import math

import numpy as np


def softmax_weights(logits: np.ndarray) -> np.ndarray:
    """Softmax over the last axis with max subtraction (definition, fp64)."""
    logits = np.asarray(logits, dtype=np.float64)
    shifted = logits - logits.max(axis=-1, keepdims=True)
    e = np.exp(shifted)
    return e / e.sum(axis=-1, keepdims=True)


def dense_decode_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """One trace, contiguous (unpaged) KV.

    q : [Hq, d]        query of the new token, all query heads
    K : [S, Hkv, d]    keys of the trace's S logical positions
    V : [S, Hkv, d]    values
    returns [Hq, d] float64
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    Hq, d = q.shape
    S, Hkv, d2 = K.shape
    assert d2 == d and V.shape == K.shape and Hq % Hkv == 0
    G = Hq // Hkv
    out = np.zeros((Hq, d), dtype=np.float64)
    if S == 0:
        return out
    inv_sqrt_d = 1.0 / math.sqrt(d)
    for h in range(Hq):
        g = h // G
        logits = (K[:, g, :] @ q[h]) * inv_sqrt_d          # [S]
        p = softmax_weights(logits)                         # [S]
        out[h] = p @ V[:, g, :]                             # [d]
    return out


def gather_trace_kv(k_pages: np.ndarray, v_pages: np.ndarray,
                    block_row: np.ndarray, seq_len: int):
    """Logical K/V sequence of one trace read through its block-table row.

    k_pages, v_pages : [num_blocks, Hkv, P, d]  one layer of the paged pool
    block_row        : [max_pages] int          physical block of each logical page
    Logical position j lives in block block_row[j // P], slot j % P.
    returns K, V : [seq_len, Hkv, d]
    """
    num_blocks, Hkv, P, d = k_pages.shape
    K = np.empty((seq_len, Hkv, d), dtype=np.float64)
    V = np.empty((seq_len, Hkv, d), dtype=np.float64)
    for page in range((seq_len + P - 1) // P):
        b = int(block_row[page])
        assert 0 <= b < num_blocks, "logical page maps to no block"
        j0 = page * P
        cnt = min(P, seq_len - j0)                 # last page may be partly filled
        # slot s of the page is logical position j0 + s
        K[j0:j0 + cnt] = np.swapaxes(k_pages[b, :, :cnt, :], 0, 1)
        V[j0:j0 + cnt] = np.swapaxes(v_pages[b, :, :cnt, :], 0, 1)
    return K, V


def paged_decode_attention(q: np.ndarray, k_pages: np.ndarray, v_pages: np.ndarray,
                           block_table: np.ndarray, seq_lens: np.ndarray) -> np.ndarray:
    """All traces of one decode step, one layer.

    q           : [n, Hq, d]
    k_pages     : [num_blocks, Hkv, P, d]
    v_pages     : [num_blocks, Hkv, P, d]
    block_table : [n, max_pages] int
    seq_lens    : [n] int
    returns [n, Hq, d] float64
    """
    q = np.asarray(q, dtype=np.float64)
    n = q.shape[0]
    out = np.zeros(q.shape, dtype=np.float64)
    for t in range(n):
        S = int(seq_lens[t])
        K, V = gather_trace_kv(k_pages, v_pages, block_table[t], S)
        out[t] = dense_decode_attention(q[t], K, V)
    return out


def paged_decode_attention_shared_prefix(q, k_pages, v_pages, block_table, seq_lens, prefix_blocks):
    """Decode attention of traces whose first len(prefix_blocks) pages are the given shared blocks.

    Trace t attends to the positions of the shared pages (in order) followed by its own positions
    [len(prefix_blocks) * P, seq_lens[t]) read through its block-table row; this is paged_decode_attention whenever
    the row's first entries equal prefix_blocks (the prompt pages all traces of one problem share: Algorithm 1,
    InitTraces).  A trace with seq_lens[t] = 0, or shorter than the prefix, yields zeros; the ids of the latter are
    returned as the second result.
    """
    q = np.asarray(q, dtype=np.float64)
    P = k_pages.shape[2]
    pp = len(prefix_blocks)
    out = np.zeros(q.shape, dtype=np.float64)
    too_short = []
    for t in range(q.shape[0]):
        S = int(seq_lens[t])
        if S == 0:
            continue
        if S < pp * P:
            too_short.append(t)
            continue
        row = np.array(block_table[t]).copy()
        row[:pp] = np.asarray(prefix_blocks)
        K, V = gather_trace_kv(k_pages, v_pages, row, S)
        out[t] = dense_decode_attention(q[t], K, V)
    return out, too_short


def merge_partials(ms, ls, os_):
    """Combine split evaluations of one softmax-weighted sum.

    Each part i covers a disjoint subset of positions and carries
      m_i = max logit in the part, l_i = sum exp(logit - m_i),
      o_i = sum exp(logit - m_i) * v   (unnormalised).
    The merged result is  sum_i e^{m_i - M} o_i / sum_i e^{m_i - M} l_i,
    M = max_i m_i.  Used by tests to state the split-evaluation identity;
    the direct functions above never call it.
    """
    ms = np.asarray(ms, dtype=np.float64)
    M = ms.max()
    w = np.exp(ms - M)
    l = float((w * np.asarray(ls, dtype=np.float64)).sum())
    o = (w[:, None] * np.asarray(os_, dtype=np.float64)).sum(axis=0)
    return o / l


def partial_of_range(qh: np.ndarray, Kg: np.ndarray, Vg: np.ndarray, lo: int, hi: int):
    """(m, l, o) of positions [lo, hi) for one head; companion of merge_partials."""
    d = qh.shape[0]
    logits = (np.asarray(Kg[lo:hi], np.float64) @ np.asarray(qh, np.float64)) / math.sqrt(d)
    m = logits.max()
    e = np.exp(logits - m)
    return m, e.sum(), e @ np.asarray(Vg[lo:hi], np.float64)


def attention_flops(Hq: int, d: int, seq_len: int) -> int:
    """2*d multiply-adds for q.k and 2*d for p.v per position per query head."""
    return 4 * Hq * d * seq_len

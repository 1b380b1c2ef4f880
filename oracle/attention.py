"""Oracle attention for a mixed CTB batch, in float64 (test infrastructure only).

What a resumed task computes (paper Section 4: a paused task resumes from its
preserved state with the observation tokens appended; Section 1, first
challenge: recomputing the history would be pure redundancy, so resuming must
give what recomputation gives).  The paper leaves the attention maths to the
inference engine; the definition used is ordinary scaled-dot-product softmax
attention with grouped KV heads:

  row b = (task, q_len n, ctx_len L); preserved prefix p = L - n
  query i in [0, n) sits at absolute position p + i and sees keys j in [0, p + i]
  (bottom-right aligned causal mask: a decode row, n = 1, sees all L keys)
  query head h reads KV head h // G, G = Hq // Hkv
  s_j = scale * <q, k_j>;  m = max_j s_j;  l = sum_j exp(s_j - m)
  O = sum_j exp(s_j - m) v_j / l;  LSE = m + ln l   (natural log, scaled logits)

bf16 inputs are widened to float64 exactly; all arithmetic is float64.
"""
from __future__ import annotations

import math

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of raw bf16 bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def attend_contiguous(q_bits, k_bits, v_bits, scale: float, q_block: int = 256):
    """One row.  q_bits [n, Hq, D], k_bits / v_bits [L, Hkv, D] (uint16 bf16 bits), L >= n.

    Returns O [n, Hq, D] float64 and LSE [n, Hq] float64."""
    n, Hq, D = q_bits.shape
    L, Hkv, _ = k_bits.shape
    assert 1 <= n <= L and Hq % Hkv == 0
    G = Hq // Hkv
    p = L - n
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    v = bf16_bits_to_f64(v_bits)
    out = np.empty((n, Hq, D), dtype=np.float64)
    lse = np.empty((n, Hq), dtype=np.float64)
    key_pos = np.arange(L)
    for h in range(Hq):
        g = h // G
        kg, vg = k[:, g, :], v[:, g, :]
        for i0 in range(0, n, q_block):
            i1 = min(n, i0 + q_block)
            s = scale * (q[i0:i1, h, :] @ kg.T)                      # [nb, L]
            visible = key_pos[None, :] <= (p + np.arange(i0, i1))[:, None]
            s = np.where(visible, s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            l = e.sum(axis=1, keepdims=True)
            out[i0:i1, h, :] = (e @ vg) / l
            lse[i0:i1, h] = (m + np.log(l))[:, 0]
    return out, lse


def attend(cache, rows, q_bits, scale: float):
    """A batch.  cache: PagedKVOracle; rows: list of (task, q_len, ctx_len);
    q_bits: uint16 [sum q_len, Hq, D], rows concatenated in batch order.

    Returns O [sum q_len, Hq, D] and LSE [sum q_len, Hq] in float64."""
    cache.check_rows(rows)
    total = sum(int(r[1]) for r in rows)
    assert q_bits.shape[0] == total
    Hq, D = q_bits.shape[1], q_bits.shape[2]
    out = np.empty((total, Hq, D), dtype=np.float64)
    lse = np.empty((total, Hq), dtype=np.float64)
    off = 0
    for (task, n, L) in rows:
        k_bits, v_bits = cache.read(int(task), int(L))
        o, e = attend_contiguous(q_bits[off:off + n], k_bits, v_bits, scale)
        out[off:off + n], lse[off:off + n] = o, e
        off += n
    return out, lse


def attend_bruteforce(q, k, v, scale: float):
    """The definition as scalar loops, for tiny inputs.  q [n, Hq, D], k / v [L, Hkv, D]
    as Python/NumPy floats (already widened).  Returns nested lists O[n][Hq][D], LSE[n][Hq]."""
    n, Hq, D = len(q), len(q[0]), len(q[0][0])
    L, Hkv = len(k), len(k[0])
    G = Hq // Hkv
    p = L - n
    O = [[[0.0] * D for _ in range(Hq)] for _ in range(n)]
    LSE = [[0.0] * Hq for _ in range(n)]
    for i in range(n):
        last = p + i
        for h in range(Hq):
            g = h // G
            s = []
            for j in range(last + 1):
                acc = 0.0
                for d in range(D):
                    acc += float(q[i][h][d]) * float(k[j][g][d])
                s.append(scale * acc)
            m = max(s)
            w = [math.exp(x - m) for x in s]
            l = math.fsum(w)
            for d in range(D):
                O[i][h][d] = math.fsum(w[j] * float(v[j][g][d]) for j in range(last + 1)) / l
            LSE[i][h] = m + math.log(l)
    return O, LSE


def attend_subset(q_vec, k, v, scale: float, key_idx):
    """Attention of ONE query vector [D] over the keys listed in key_idx (possibly empty).
    Returns (O [D], LSE); an empty subset gives (zeros, -inf)."""
    D = q_vec.shape[0]
    key_idx = np.asarray(key_idx, dtype=np.int64)
    if key_idx.size == 0:
        return np.zeros(D), -np.inf
    s = scale * (k[key_idx] @ q_vec)
    m = s.max()
    e = np.exp(s - m)
    l = e.sum()
    return (e @ v[key_idx]) / l, m + math.log(l)


def merge(partial_o, partial_lse):
    """Log-sum-exp merge of attention over disjoint key subsets.

    partial_o [k, D], partial_lse [k]; LSE = ln sum_i exp(LSE_i),
    O = sum_i exp(LSE_i - LSE) O_i; a subset with LSE_i = -inf weighs 0."""
    partial_o = np.asarray(partial_o, dtype=np.float64)
    partial_lse = np.asarray(partial_lse, dtype=np.float64)
    top = partial_lse.max()
    if not np.isfinite(top):
        return np.zeros(partial_o.shape[1]), -np.inf
    w = np.exp(partial_lse - top)
    tot = w.sum()
    lse = top + math.log(tot)
    o = (w[:, None] * partial_o).sum(axis=0) / tot
    return o, lse

"""CPU oracle: logits over the static vocabulary joined with one sequence's hypertokens, and the
reductions taken from them, in fp64 (TEST INFRASTRUCTURE ONLY).

Section 2.3, steps 7-9: the hyper-unembedding rows of a sequence are appended to the static
unembedding matrix, a joint softmax is taken over the union vocabulary, and a token (base or
hyper) is selected.  Written out as the plain definition:

    l_j      = <W_U[j], h>            j <  V
    l_{V+i}  = <U_h[b][i], h>         i <  n_vis   (rows of the sequence that owns h)
    LSE      = m + log(sum_j exp(l_j - m)),   m = max_j l_j
    argmax   = lowest j attaining m

Sampling uses the Gumbel-max identity: argmax_j (l_j / T + g_j), g_j = -log(-log u_j), is a draw
from softmax(l / T).  u_j comes from the counter-based generator Philox4x32-10 (Salmon et al.,
SC'11) keyed by the seed, with counter (j // 4, row, step_lo, step_hi) and output word j % 4,
mapped to the open unit interval as ((x >> 9) + 0.5) * 2^-23 so that the value is exact in fp32.

Pins: tests/test_oracle_logits.py (Philox known-answer vectors from the generator's publication;
sum_j exp(l_j - LSE) == 1; with no hypertokens equals an ordinary LM head via a library matmul;
LSE over the union >= LSE over the static part; Gumbel-max frequencies approach softmax).
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32 on arrays of counters (uint32 each); returns four uint32 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK
    k0 &= 0xFFFFFFFF
    k1 &= 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0                      # 32x32 -> 64-bit products
        p1 = _M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK
        n0 = hi1 ^ c1 ^ np.uint64(k0)
        n2 = hi0 ^ c3 ^ np.uint64(k1)
        c0, c1, c2, c3 = n0, lo1, n2, lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def uniform_open(j: np.ndarray, row: int, step: int, seed: int) -> np.ndarray:
    """u_j in (0,1) for column indices ``j`` of one row at one step."""
    j = np.asarray(j, dtype=np.uint64)
    words = philox4x32_10(j >> np.uint64(2), np.full(j.shape, row, dtype=np.uint64),
                          np.full(j.shape, step & 0xFFFFFFFF, dtype=np.uint64),
                          np.full(j.shape, (step >> 32) & 0xFFFFFFFF, dtype=np.uint64),
                          seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    w = np.stack(words, axis=0)                       # [4, n]
    x = w[(j & np.uint64(3)).astype(np.int64), np.arange(j.shape[0])]
    return ((x >> np.uint32(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def gumbel(j: np.ndarray, row: int, step: int, seed: int) -> np.ndarray:
    return -np.log(-np.log(uniform_open(j, row, step, seed)))


def joint_logits(h: np.ndarray, W_U: np.ndarray, U_h_rows: Optional[np.ndarray]) -> np.ndarray:
    """All logits of one hidden state: static part then the visible hypertoken rows."""
    l = W_U @ h
    if U_h_rows is not None and U_h_rows.shape[0] > 0:
        l = np.concatenate([l, U_h_rows @ h])
    return l


def lse(l: np.ndarray) -> float:
    m = float(l.max())
    return m + float(np.log(np.exp(l - m).sum()))


def top2(l: np.ndarray) -> Tuple[int, float, float]:
    """(argmax with lowest-index tie rule, its value, gap to the best OTHER index)."""
    a = int(np.argmax(l))                 # numpy returns the first maximum
    best = float(l[a])
    if l.shape[0] == 1:
        return a, best, float("inf")
    rest = np.delete(l, a)
    return a, best, best - float(rest.max())


def select(l: np.ndarray, mode: int, temperature: float, seed: int, step: int, row: int):
    """Token selection.  mode 0: argmax; mode 1: Gumbel-max sample at ``temperature``.
    Returns (choice, scores, gap) where ``scores`` are the values the decision was taken on."""
    if mode == 0:
        scores = l
    else:
        scores = l / float(temperature) + gumbel(np.arange(l.shape[0]), row, step, seed)
    a, _, gap = top2(scores)
    return a, scores, gap


def filter_mask(l: np.ndarray, temperature: float, top_k: int, top_p: float) -> np.ndarray:
    """Columns that top-k and nucleus (top-p) filtering keep.  Neither is defined by the paper,
    which only says that a token is sampled from the joint distribution (Section 2.3 step 9);
    these are the usual definitions, with ties kept together so that the result does not depend
    on an order among equal logits:
      top-k: every column whose logit is >= the k-th largest logit (top_k <= 0: no filter);
      top-p: with columns in descending order of probability softmax(l / T), the shortest prefix
             whose probabilities sum to >= top_p, extended over ties with its last logit
             (top_p >= 1: no filter).
    The result is the intersection; the argmax is always kept."""
    l = np.asarray(l, dtype=np.float64)
    n = l.shape[0]
    keep = np.ones(n, dtype=bool)
    if 0 < top_k < n:
        vk = np.sort(l)[::-1][top_k - 1]
        keep &= l >= vk
    if top_p < 1.0:
        order = np.argsort(-l, kind="stable")
        ls = l[order]
        pr = np.exp((ls - ls[0]) / float(temperature))
        cum = np.cumsum(pr) / pr.sum()
        j = int(np.searchsorted(cum, top_p, side="left"))
        j = min(j, n - 1)
        keep &= l >= ls[j]
    return keep


def select_filtered(l: np.ndarray, temperature: float, top_k: int, top_p: float, seed: int, step: int, row: int):
    """Gumbel-max sample from softmax(l / T) restricted to filter_mask (the noise of a column does
    not depend on the filter).  Returns (choice, kept mask, gap between the two best kept scores)."""
    keep = filter_mask(l, temperature, top_k, top_p)
    scores = np.asarray(l, dtype=np.float64) / float(temperature) + gumbel(np.arange(l.shape[0]), row, step, seed)
    scores = np.where(keep, scores, -np.inf)
    a, _, gap = top2(scores)
    return a, keep, gap

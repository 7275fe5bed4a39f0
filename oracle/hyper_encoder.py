"""CPU oracle: the hyper-encoder f_phi in fp64 (TEST INFRASTRUCTURE ONLY).

Section 2.2 defines f_phi : V^M -> R^d as a network over the embeddings of a hypertoken's
constituent base tokens, inputs padded to M; Section 3.1 fixes it to a two-layer transformer
encoder; the appendix on hyper-encoder architecture lists the parameter-free "averaging" variant
as the zero-layer case.  The paper does not spell the layer out, so this file writes down the
textbook pre-LayerNorm encoder layer (the reading is listed in the design notes):

    X_i = W[y_i] + pos_i                                 i = 1..L   (L <= M valid positions)
    for each layer:
        A = LN1(X);  Q,K,V = A Wq^T + bq, A Wk^T + bk, A Wv^T + bv     (packed Wqkv, bqkv)
        per head h: P = softmax(Q_h K_h^T / sqrt(d/H)) over the L valid keys;  O_h = P V_h
        X = X + concat(O_h) Wo^T + bo
        X = X + W2 gelu(W1 LN2(X) + b1) + b2             (erf GELU; LayerNorm eps 1e-5)
    h = mean_i X_i                                       over the L valid positions

A layer whose feed-forward width is zero (W1 has no rows) is the attention sublayer alone: with one
such layer this is the "1-attention-layer" variant of the appendix's architecture ablation (read
as the first sublayer of the same pre-LN layer, residual included; the paper gives no detail).

Padding positions are never used as keys and never pooled, so their values cannot matter and are
not computed.  Everything is numpy fp64 on the exact values of the (bf16 or fp32) inputs.

Pins: tests/test_oracle_encoder.py (zero layers == plain mean of the gathered rows; one and two
layers against torch.nn.TransformerEncoderLayer(norm_first=True) with a key-padding mask;
permutation sensitivity through ``pos``; attention-only layers against
torch.nn.MultiheadAttention on LayerNorm'd rows, and == plain mean when Wo and bo are zero).  The absolute values under the paper's *trained*
encoder are "parity unpinned": no weights exist offline.
"""
from __future__ import annotations

import math
from typing import List, Sequence

import numpy as np
from scipy.special import erf as _erf

LN_EPS = 1e-5
PER_LAYER = 12     # ln1_w ln1_b Wqkv bqkv Wo bo ln2_w ln2_b W1 b1 W2 b2


def _layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + LN_EPS) * g + b


def _gelu(x: np.ndarray) -> np.ndarray:
    """Exact (erf) GELU: x * Phi(x)."""
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def hyper_embed_one(constituents: Sequence[int], table: np.ndarray, enc: List[np.ndarray],
                    heads: int) -> np.ndarray:
    """f_phi for one hypertoken.  ``table`` is W_E (or W_U) as fp64 ``[V, d]``; ``enc`` is the
    tensor list ``[pos, (12 tensors per layer)...]`` as fp64 arrays."""
    y = [int(t) for t in constituents]
    L = len(y)
    d = table.shape[1]
    pos = enc[0]
    X = table[y, :] + pos[:L, :]                                  # [L, d]
    n_layers = (len(enc) - 1) // PER_LAYER
    dh = d // heads
    for l in range(n_layers):
        (ln1_w, ln1_b, Wqkv, bqkv, Wo, bo, ln2_w, ln2_b, W1, b1, W2, b2) = \
            enc[1 + l * PER_LAYER: 1 + (l + 1) * PER_LAYER]
        A = _layer_norm(X, ln1_w, ln1_b)
        qkv = A @ Wqkv.T + bqkv                                   # [L, 3d]
        Q, K, Vv = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
        O = np.empty_like(Q)
        for h in range(heads):
            s = slice(h * dh, (h + 1) * dh)
            S = (Q[:, s] @ K[:, s].T) / math.sqrt(dh)             # [L, L], all keys valid
            S = S - S.max(axis=1, keepdims=True)
            P = np.exp(S)
            P = P / P.sum(axis=1, keepdims=True)
            O[:, s] = P @ Vv[:, s]
        X = X + O @ Wo.T + bo
        if W1.shape[0] == 0:                                      # attention-only layer
            continue
        Hh = _gelu(_layer_norm(X, ln2_w, ln2_b) @ W1.T + b1)
        X = X + Hh @ W2.T + b2
    return X.mean(axis=0)


def hyper_embed(entries: Sequence[Sequence[int]], table: np.ndarray, enc: List[np.ndarray],
                heads: int) -> np.ndarray:
    """Rows of the hyper-embedding cache for a list of codebook entries: ``[len(entries), d]``.

    Same function as ``hyper_embed_one`` applied to each entry.  The only difference is that the
    position-wise maps (LayerNorm, the four linear layers, GELU) are applied to the valid rows of
    all entries stacked into one matrix, so that each fp64 weight matrix is read once per call
    instead of once per entry; attention and pooling stay per entry.  A test checks that the two
    agree to rounding.
    """
    d = table.shape[1]
    if len(entries) == 0:
        return np.empty((0, d), dtype=np.float64)
    pos = enc[0]
    lens = [len(e) for e in entries]
    offs = np.concatenate([[0], np.cumsum(lens)])
    ids = np.concatenate([np.asarray(e, dtype=np.int64) for e in entries])
    pidx = np.concatenate([np.arange(L) for L in lens])
    X = table[ids, :] + pos[pidx, :]
    n_layers = (len(enc) - 1) // PER_LAYER
    dh = d // heads
    for l in range(n_layers):
        (ln1_w, ln1_b, Wqkv, bqkv, Wo, bo, ln2_w, ln2_b, W1, b1, W2, b2) = \
            enc[1 + l * PER_LAYER: 1 + (l + 1) * PER_LAYER]
        qkv = _layer_norm(X, ln1_w, ln1_b) @ Wqkv.T + bqkv
        O = np.empty((X.shape[0], d), dtype=np.float64)
        for e in range(len(entries)):
            r = slice(offs[e], offs[e + 1])
            for h in range(heads):
                s = slice(h * dh, (h + 1) * dh)
                S = (qkv[r, s] @ qkv[r, d + h * dh: d + (h + 1) * dh].T) / math.sqrt(dh)
                S = S - S.max(axis=1, keepdims=True)
                P = np.exp(S)
                P = P / P.sum(axis=1, keepdims=True)
                O[r, s] = P @ qkv[r, 2 * d + h * dh: 2 * d + (h + 1) * dh]
        X = X + O @ Wo.T + bo
        if W1.shape[0] == 0:                                      # attention-only layer
            continue
        X = X + _gelu(_layer_norm(X, ln2_w, ln2_b) @ W1.T + b1) @ W2.T + b2
    out = np.empty((len(entries), d), dtype=np.float64)
    for e in range(len(entries)):
        out[e] = X[offs[e]:offs[e + 1]].mean(axis=0)
    return out

"""Seeded synthetic inputs for the dynamic-vocabulary path (token streams, weights, hidden states).

This module holds NO arithmetic of the method itself (no LZW, no encoder, no logits): it only
draws numbers.  Both the CUDA path and the CPU oracle consume the arrays it returns, so that the
two never share anything else.

The token streams stand in for the paper's corpora (Section 3, Table "token_efficiency"), which
need tokenizers and datasets that are not available offline: base tokens follow a Zipf law over a
seeded permutation of the vocabulary, and with probability ``copy_p`` a position starts a verbatim
copy of an earlier segment, so that recurring n-grams exist and hypertokens form.  Weights are
N(0, 0.02) and hidden states N(0, 1), rounded to the storage dtype: the rounded values ARE the
inputs on both sides.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration (shapes and generator parameters)."""
    name: str
    V: int            # static vocabulary size
    d: int            # embedding dimension
    dtype: str        # "fp32" or "bf16": storage type of weights, hidden states and caches
    B: int            # sequences
    T: int            # prompt tokens per sequence
    M: int            # maximum merge size (Section 2.1)
    cap: int          # maximum hypertokens per sequence
    zipf_s: float
    copy_p: float
    seg_min: int
    seg_max: int
    steps: int        # decode steps (0: prefill-only workload)
    enc_layers: int = 2       # "two-layer transformer encoder" (Section 3.1)
    enc_heads: int = 0        # 0 -> d // 128 (tiny: 4)
    enc_dff: int = 0          # 0 -> 4 * d
    tied: int = 0
    enc_ffn: int = 1          # 0: attention-only layers (feed-forward width 0; architecture ablation)

    @property
    def heads(self) -> int:
        if self.enc_heads:
            return self.enc_heads
        return max(1, self.d // 128) if self.d >= 128 else 4

    @property
    def dff(self) -> int:
        if not self.enc_ffn:
            return 0
        return self.enc_dff if self.enc_dff else 4 * self.d

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations of the benchmark definition, in its order.
WORKLOADS: Dict[str, Workload] = {
    "tiny": Workload("tiny", V=512, d=64, dtype="fp32", B=1, T=256, M=3, cap=256,
                     zipf_s=1.1, copy_p=0.3, seg_min=4, seg_max=16, steps=64),
    "phi3_mini_head": Workload("phi3_mini_head", V=32064, d=3072, dtype="bf16", B=8, T=2048, M=3,
                               cap=2048, zipf_s=1.1, copy_p=0.3, seg_min=4, seg_max=16, steps=256),
    "llama3_8b_head": Workload("llama3_8b_head", V=128256, d=4096, dtype="bf16", B=32, T=4096, M=3,
                               cap=4096, zipf_s=1.2, copy_p=0.4, seg_min=4, seg_max=32, steps=512),
    "prefill_heavy": Workload("prefill_heavy", V=128256, d=4096, dtype="bf16", B=64, T=8192, M=4,
                              cap=8192, zipf_s=1.2, copy_p=0.4, seg_min=4, seg_max=32, steps=0),
    "long_context": Workload("long_context", V=128256, d=4096, dtype="bf16", B=4, T=32768, M=5,
                             cap=16384, zipf_s=1.0, copy_p=0.6, seg_min=8, seg_max=64, steps=1024),
}


def _zipf_cdf(V: int, s: float) -> np.ndarray:
    w = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    c = np.cumsum(w)
    return c / c[-1]


def token_stream(V: int, T: int, zipf_s: float, copy_p: float, seg_min: int, seg_max: int,
                 seed: int) -> np.ndarray:
    """One sequence of ``T`` base-token ids in ``[0, V)``.

    Outside a copy, a position starts (with probability ``copy_p``, once at least ``seg_min``
    tokens of history exist) a verbatim copy of ``len ~ U{seg_min..seg_max}`` tokens from a
    uniformly chosen earlier start; otherwise it draws rank ~ Zipf(s) and maps it through a seeded
    permutation of the vocabulary.
    """
    rng = np.random.Generator(np.random.Philox(key=int(seed) & 0xFFFFFFFFFFFFFFFF))
    perm = rng.permutation(V).astype(np.int32)
    cdf = _zipf_cdf(V, zipf_s)
    ranks = np.searchsorted(cdf, rng.random(T), side="left").clip(0, V - 1)
    fresh = perm[ranks]
    coin = rng.random(T)
    seg_len = rng.integers(seg_min, seg_max + 1, size=T)
    start_u = rng.random(T)
    out = np.empty(T, dtype=np.int32)
    t = 0
    while t < T:
        if t >= seg_min and coin[t] < copy_p:
            ln = int(min(seg_len[t], T - t, t))
            src = int(start_u[t] * (t - ln + 1))
            # source and destination may not overlap: src + ln <= t
            out[t:t + ln] = out[src:src + ln]
            t += ln
        else:
            out[t] = fresh[t]
            t += 1
    return out


def make_tokens(w: Workload, seed: int, T: int | None = None) -> np.ndarray:
    """``[B, T]`` int32 prompt tokens; sequence ``b`` uses seed ``seed * 1000003 + b``."""
    T = w.T if T is None else T
    return np.stack([token_stream(w.V, T, w.zipf_s, w.copy_p, w.seg_min, w.seg_max,
                                  seed * 1000003 + b) for b in range(w.B)])


def normal_tensor(shape, std: float, seed: int, dtype: torch.dtype) -> torch.Tensor:
    """N(0, std) values drawn in fp32 on the CPU and rounded (RNE) to ``dtype``."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    n = 1
    for s in shape:
        n *= int(s)
    # draw in chunks so very large tables do not need a second full fp32 copy
    out = torch.empty(n, dtype=dtype)
    chunk = 1 << 24
    for i in range(0, n, chunk):
        m = min(chunk, n - i)
        out[i:i + m] = (torch.randn(m, generator=g, dtype=torch.float32) * std).to(dtype)
    return out.view(*shape)


# Order of the hyper-encoder tensors, shared by the ABI and by the oracle's argument list:
#   pos[M,d], then per layer:
#   ln1_w[d] ln1_b[d] Wqkv[3d,d] bqkv[3d] Wo[d,d] bo[d] ln2_w[d] ln2_b[d] W1[dff,d] b1[dff] W2[d,dff] b2[d]
ENC_TENSORS_PER_LAYER = 12


def encoder_shapes(w: Workload) -> List[tuple]:
    d, dff = w.d, w.dff
    shapes = [("pos", (w.M, d))]
    for l in range(w.enc_layers):
        shapes += [(f"l{l}.ln1_w", (d,)), (f"l{l}.ln1_b", (d,)),
                   (f"l{l}.Wqkv", (3 * d, d)), (f"l{l}.bqkv", (3 * d,)),
                   (f"l{l}.Wo", (d, d)), (f"l{l}.bo", (d,)),
                   (f"l{l}.ln2_w", (d,)), (f"l{l}.ln2_b", (d,)),
                   (f"l{l}.W1", (dff, d)), (f"l{l}.b1", (dff,)),
                   (f"l{l}.W2", (d, dff)), (f"l{l}.b2", (d,))]
    return shapes


def make_encoder(w: Workload, seed: int, *, generic: bool = False) -> List[torch.Tensor]:
    """Hyper-encoder tensors in ABI order.

    Default init follows the benchmark definition: matrices and ``pos`` ~ N(0, 0.02), LayerNorm
    gain 1 / bias 0, linear biases 0.  ``generic=True`` draws every gain and bias at random too, so
    that parity tests exercise those terms.
    """
    out = []
    for i, (name, shape) in enumerate(encoder_shapes(w)):
        leaf = name.split(".")[-1]
        if leaf in ("ln1_w", "ln2_w") and not generic:
            t = torch.ones(shape, dtype=w.torch_dtype)
        elif leaf in ("ln1_w", "ln2_w"):
            t = (1.0 + normal_tensor(shape, 0.1, seed * 131 + i, torch.float32)).to(w.torch_dtype)
        elif leaf in ("ln1_b", "ln2_b", "bqkv", "bo", "b1", "b2") and not generic:
            t = torch.zeros(shape, dtype=w.torch_dtype)
        elif leaf in ("ln1_b", "ln2_b", "bqkv", "bo", "b1", "b2"):
            t = normal_tensor(shape, 0.05, seed * 131 + i, w.torch_dtype)
        else:
            t = normal_tensor(shape, 0.02, seed * 131 + i, w.torch_dtype)
        out.append(t)
    return out


def make_tables(w: Workload, seed: int):
    """Static embedding / unembedding tables ``W_E``, ``W_U`` of shape ``[V, d]``."""
    W_E = normal_tensor((w.V, w.d), 0.02, seed * 7 + 1, w.torch_dtype)
    W_U = W_E if w.tied else normal_tensor((w.V, w.d), 0.02, seed * 7 + 2, w.torch_dtype)
    return W_E, W_U


def make_hidden(w: Workload, n_rows: int, seed: int) -> torch.Tensor:
    """``[n_rows, d]`` hidden states ~ N(0, 1) in the storage dtype."""
    return normal_tensor((n_rows, w.d), 1.0, seed * 7 + 3, w.torch_dtype)

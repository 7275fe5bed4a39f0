"""CPU oracle: one whole decode step of the dynamic-vocabulary path (TEST INFRASTRUCTURE ONLY).

Section 2.3 in the paper's order: logits over V u V_h and token selection (steps 7-9), the online
LZW update with the selected token (step 10, "created at step t, usable at t+1"), then the
hyper-encoder on the at most one new entry per sequence, for the embedding-side and the
unembedding-side cache alike ("Hyper-Embedding Cache": one new hypertoken per step; "Consistent
Vocabulary Updates": both sides see the same hypertoken set).

``score`` does the first part without touching state; ``advance`` does the rest with whatever
code the caller passes.  Keeping them apart lets a parity test follow the GPU's selection where
the oracle's own top-2 gap is below the stated threshold (several answers are then correct).

Caches hold what the storage type can represent: fp64 results are rounded to bf16 (round to
nearest even) or fp32 before they are stored, because the logits of later steps are defined on
the stored rows.  The unrounded fp64 rows are kept beside them for checking the encoder alone.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

from . import hyper_encoder, logits as lg, lzw


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64 values to the cache's storage type and return them as fp64."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    if dtype == "fp32":
        return f.astype(np.float64)
    bits = f.view(np.uint32).astype(np.uint64)
    # bf16 keeps the top 16 bits of the fp32 pattern; round to nearest, ties to even
    bits = bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1))
    bits = (bits >> np.uint64(16)) << np.uint64(16)
    return bits.astype(np.uint32).view(np.float32).astype(np.float64)


class Session:
    """All sequences of one inference session: codebooks and both caches."""

    def __init__(self, V: int, M: int, cap: int, B: int, heads: int, dtype: str,
                 W_E: np.ndarray, W_U: np.ndarray, enc_E: List[np.ndarray],
                 enc_U: List[np.ndarray]):
        self.V, self.M, self.cap, self.B, self.heads, self.dtype = V, M, cap, B, heads, dtype
        self.W_E, self.W_U, self.enc_E, self.enc_U = W_E, W_U, enc_E, enc_U
        d = W_U.shape[1]
        self.books = [lzw.Codebook(V, M, cap) for _ in range(B)]
        self.E_h = [np.empty((0, d)) for _ in range(B)]        # stored (rounded) rows
        self.U_h = [np.empty((0, d)) for _ in range(B)]
        self.E_exact = [np.empty((0, d)) for _ in range(B)]    # unrounded fp64 rows
        self.U_exact = [np.empty((0, d)) for _ in range(B)]

    # -- prefill: compress each prompt, embed every entry it created -------------------------
    def prefill(self, prompts: Sequence[Sequence[int]]):
        codes, after = [], []
        for b, x in enumerate(prompts):
            c, a = self.books[b].encode(x)
            codes.append(c)
            after.append(a)
            self._embed_new(b)
        return codes, after

    def _embed_new(self, b: int):
        have = self.E_h[b].shape[0]
        new = self.books[b].entries[have:]
        if not new:
            return
        e = hyper_encoder.hyper_embed(new, self.W_E, self.enc_E, self.heads)
        u = hyper_encoder.hyper_embed(new, self.W_U, self.enc_U, self.heads)
        self.E_exact[b] = np.concatenate([self.E_exact[b], e])
        self.U_exact[b] = np.concatenate([self.U_exact[b], u])
        self.E_h[b] = np.concatenate([self.E_h[b], round_to_storage(e, self.dtype)])
        self.U_h[b] = np.concatenate([self.U_h[b], round_to_storage(u, self.dtype)])

    # -- steps 7-9: joint logits and selection (no state change) ------------------------------
    def score(self, hidden: np.ndarray, mode: int = 0, temperature: float = 1.0, seed: int = 0,
              step: int = 0):
        """For each sequence b (row b of ``hidden``): dict with the joint logits ``l``, ``lse``,
        the oracle's ``choice``, the decision ``scores`` and the top-2 ``gap`` on them."""
        out = []
        for b in range(self.B):
            l = lg.joint_logits(hidden[b], self.W_U, self.U_h[b])
            choice, scores, gap = lg.select(l, mode, temperature, seed, step, b)
            out.append({"l": l, "lse": lg.lse(l), "choice": choice, "scores": scores, "gap": gap})
        return out

    # -- step 10 + cache update ---------------------------------------------------------------
    def advance(self, codes: Sequence[int], active: Optional[Sequence[bool]] = None):
        """Apply the selected codes: LZW update, then embed the new entry (if any) on both
        sides.  Returns the new entry number per sequence (-1 if none)."""
        new = []
        for b in range(self.B):
            if active is not None and not active[b]:
                new.append(-1)
                continue
            k = self.books[b].step(int(codes[b]))
            new.append(k)
            if k >= 0:
                self._embed_new(b)
        return new

    def step(self, hidden: np.ndarray, mode: int = 0, temperature: float = 1.0, seed: int = 0,
             step: int = 0):
        """O5: score, select, advance with the oracle's own choices."""
        sc = self.score(hidden, mode, temperature, seed, step)
        new = self.advance([s["choice"] for s in sc])
        return sc, new

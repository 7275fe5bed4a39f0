"""CPU oracle: LZW over base-token ids with a maximum merge size (TEST INFRASTRUCTURE ONLY).

This is the plain, slow, obviously-correct statement of what the paper's tokenizer computes
(Section 2.1 "LZW Algorithm"; Figure 1 caption for ids and the "created at step t, usable at
t+1" rule; Section 2.3 steps 2 and 10-12).  It is used by tests, by the smoke check and by the
benchmark's CPU-baseline leg; the product path never imports it.  It shares no code with the CUDA
path: the codebook here is a dict keyed by the *content* of a phrase (a tuple of base tokens),
whereas the GPU keeps a hash keyed by (prefix code, next token).

Conventions (the paper leaves these open; the readings are listed in the design notes):
  * hypertoken id = V + k, k = creation order, starting at 0 (Figure 1: ids start after the
    static vocabulary);
  * a new entry is  w ++ c  (Welch's LZW, which the paper names): the phrase just emitted plus
    the single base token that follows it;
  * entries longer than M base tokens are never created (Section 2.1, "maximum merge size M");
  * at ``cap`` entries the codebook freezes: matching continues, inserting stops.

Pins: tests/test_oracle_lzw.py (worked example after Figure 1, round trip, prefix property,
bounds, replay equivalence, brute-force longest-match check on tiny vocabularies; expand()
against the self-contained decode and the original tokens).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

BAD_TOKEN = 2     # status bit: a code that names no existing (or about-to-exist) hypertoken
CAP_FROZEN = 1    # status bit: the codebook is full; informational


class Codebook:
    """Per-sequence dynamic vocabulary V_h (Section 2.2: starts empty for each session)."""

    def __init__(self, V: int, M: int, cap: int):
        self.V, self.M, self.cap = int(V), int(M), int(cap)
        self.index: Dict[Tuple[int, ...], int] = {}     # phrase content -> entry number k
        self.entries: List[Tuple[int, ...]] = []        # k -> phrase content
        self.prev: Optional[int] = None                 # last code seen by the online update
        self.status = 0

    # -- lookups ------------------------------------------------------------------------------
    def n(self) -> int:
        return len(self.entries)

    def phrase(self, code: int) -> Tuple[int, ...]:
        """Base tokens a code stands for: itself if it is a base token."""
        if 0 <= code < self.V:
            return (code,)
        return self.entries[code - self.V]

    def code_of(self, phrase: Tuple[int, ...]) -> int:
        if len(phrase) == 1:
            return phrase[0]
        return self.V + self.index[phrase]

    def _insert(self, phrase: Tuple[int, ...]) -> int:
        k = len(self.entries)
        self.index[phrase] = k
        self.entries.append(phrase)
        if len(self.entries) >= self.cap:
            self.status |= CAP_FROZEN
        return k

    # -- O1: compress a whole prompt ----------------------------------------------------------
    def encode(self, x: Sequence[int]) -> Tuple[List[int], List[int]]:
        """Greedy longest-match parse of ``x`` against the growing codebook (Section 2.1).

        Returns ``(codes, entries_after)``: ``entries_after[i]`` is the number of hypertokens that
        exist once ``codes[i]`` has been emitted (the ones a model at compressed position i+1
        could use).  Continues from the current codebook; ``prev`` is left at the last code so
        that online updates (``step``) can follow.
        """
        out: List[int] = []
        after: List[int] = []
        w: Tuple[int, ...] = ()
        for c in x:
            c = int(c)
            if not w:
                w = (c,)
                continue
            if len(w) < self.M and (w + (c,)) in self.index:
                w = w + (c,)                      # keep extending the match
                continue
            out.append(self.code_of(w))           # longest match ends here
            if len(w) < self.M and len(self.entries) < self.cap:
                self._insert(w + (c,))            # absent by construction
            after.append(len(self.entries))
            w = (c,)
        if w:
            out.append(self.code_of(w))           # final flush adds no entry
            after.append(len(self.entries))
        if out:
            self.prev = out[-1]
        return out, after

    # -- O2: online update with one newly selected code ---------------------------------------
    def step(self, z: int) -> int:
        """Decoder-side LZW update after the model emitted code ``z`` (Section 2.3, step 10).

        The candidate entry is  phrase(prev) ++ first(phrase(z)).  It is created if phrase(prev)
        is shorter than M, the codebook is not full and the phrase is not there yet.  Returns the
        new entry number, or -1.  ``z == V + n`` is the classic LZW special case (a code that
        refers to the entry this very step creates); any other id >= V + n names a hypertoken
        that does not exist (Section 2.3, "Consistent Vocabulary Updates") and leaves the state
        untouched with BAD_TOKEN set.
        """
        z = int(z)
        n = len(self.entries)
        if z < 0 or z > self.V + n:
            self.status |= BAD_TOKEN
            return -1
        if z == self.V + n:
            ok = (self.prev is not None and len(self.phrase(self.prev)) < self.M
                  and n < self.cap)
            if ok:
                p = self.phrase(self.prev)
                ok = (p + (p[0],)) not in self.index
            if not ok:
                self.status |= BAD_TOKEN
                return -1
            first = self.phrase(self.prev)[0]
        else:
            first = self.phrase(z)[0]
        new = -1
        if self.prev is not None:
            p = self.phrase(self.prev)
            if len(p) < self.M and n < self.cap and (p + (first,)) not in self.index:
                new = self._insert(p + (first,))
        self.prev = z
        return new


def encode(x: Sequence[int], V: int, M: int, cap: int):
    """Convenience: fresh codebook, compress ``x``; returns (codes, entries_after, codebook)."""
    cb = Codebook(V, M, cap)
    codes, after = cb.encode(x)
    return codes, after, cb


def decode(codes: Sequence[int], V: int, M: int, cap: int):
    """O2': rebuild the base tokens from the compressed stream alone (Section 2.1, property 2;
    Section 2.3, steps 11-12).  The decoder grows its own codebook by replaying ``step``; the
    phrase is read after the update so that the special-case id resolves.  Returns
    (tokens, codebook)."""
    cb = Codebook(V, M, cap)
    toks: List[int] = []
    for z in codes:
        cb.step(z)
        if cb.status & BAD_TOKEN:
            raise ValueError(f"code {z} names no hypertoken")
        toks.extend(cb.phrase(int(z)))
    return toks, cb


def expand(cb: Codebook, codes: Sequence[int]):
    """Codes -> base tokens with a codebook that already holds every entry (the state at the end
    of generation; Section 2.3 steps 11-12).  The codebook is not changed.  Stops before the
    first code that names no entry; returns (tokens, number of codes expanded)."""
    toks: List[int] = []
    done = 0
    for z in codes:
        z = int(z)
        if z < 0 or z >= cb.V + cb.n():
            break
        toks.extend(cb.phrase(z))
        done += 1
    return toks, done


def base_token_count(cb: Codebook, codes: Sequence[int]) -> int:
    """Number of base tokens a code sequence stands for (the 'base-token equivalent')."""
    return sum(len(cb.phrase(int(z))) for z in codes)

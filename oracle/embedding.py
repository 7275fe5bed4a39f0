"""CPU oracle: input embedding of a mixed base-token / hypertoken stream (TEST INFRASTRUCTURE ONLY).

Figure 2a and Section 2.3 steps 3-4: a base token is embedded by its row of the embedding matrix
W_E, a hypertoken by the hyper-embedding that the hyper-encoder produced for its constituents and
that the session cached (Section 2.3, "hyper-embedding cache").  The product path never imports
this module.

Pins: tests/test_oracle_lzw.py::test_lookup_* (a hypertoken's row under the parameter-free
averaging encoder equals the mean of the looked-up rows of the base tokens the LZW oracle
decompresses it to; a stream of base tokens alone reduces to numpy's row gather).
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np


def lookup(codes: Sequence[int], row_seq: Optional[Sequence[int]], W_E: np.ndarray, E_h: np.ndarray,
           n: Sequence[int]):
    """Row r of the result embeds codes[r] for sequence b = row_seq[r] (r itself if row_seq is
    None).  W_E is [V, d]; E_h is [B, cap, d]; n[b] is the number of hypertokens sequence b has.
    A code outside [0, V + n[b]) gives a zero row and is reported in the returned list ``bad``
    (sequence numbers); -1 stands for "no token" (a sequence that has finished): a zero row,
    not reported."""
    V, d = W_E.shape
    out = np.zeros((len(codes), d), dtype=np.float64)
    bad = []
    for r, z in enumerate(codes):
        z = int(z)
        b = int(row_seq[r]) if row_seq is not None else r
        if 0 <= z < V:
            out[r] = W_E[z]
        elif V <= z < V + int(n[b]):
            out[r] = E_h[b, z - V]
        elif z != -1:
            bad.append(b)
    return out, bad

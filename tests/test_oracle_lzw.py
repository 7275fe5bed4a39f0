"""Pins for oracle/lzw.py: nothing here calls the CUDA path.

Each check is chosen so that a plausible mistake in the oracle (wrong id base, inserting the
wrong phrase, ignoring M or cap, mishandling the same-step special case) fails at least one.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import lzw
from paper_2506_01084_b200 import synth_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fig1_to_be_or_not_to_be.txt")


def _golden_cases():
    cases = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, toks, codes, ents = [p.strip() for p in line.split("|")]
        V, M, cap = map(int, head.split())
        entries = {}
        for e in ents.split():
            k, v = e.split(":")
            entries[int(k)] = tuple(int(t) for t in v.split(","))
        cases.append((V, M, cap, [int(t) for t in toks.split()], [int(c) for c in codes.split()],
                      entries))
    return cases


@pytest.mark.parametrize("case", _golden_cases())
def test_worked_example_after_figure_1(case):
    V, M, cap, toks, codes, entries = case
    got, after, cb = lzw.encode(toks, V, M, cap)
    assert got == codes
    assert {V + k: e for k, e in enumerate(cb.entries)} == entries
    assert after[-1] == len(entries)
    back, cb2 = lzw.decode(got, V, M, cap)
    assert back == toks


def _streams():
    w = si.WORKLOADS["tiny"]
    out = [(w.V, si.token_stream(w.V, 600, 1.1, 0.3, 4, 16, 11))]
    out.append((50, si.token_stream(50, 2000, 1.0, 0.6, 8, 64, 12)))
    out.append((3, si.token_stream(3, 500, 1.0, 0.2, 2, 5, 13)))
    out.append((7, np.zeros(300, dtype=np.int32)))               # one symbol repeated
    out.append((7, np.arange(300, dtype=np.int32) % 7))          # short period
    return out


@pytest.mark.parametrize("M", [1, 2, 3, 5])
@pytest.mark.parametrize("cap", [0, 1, 17, 100000])
def test_round_trip_bounds_and_replay(M, cap):
    for V, x in _streams():
        x = [int(t) for t in x]
        codes, after, cb = lzw.encode(x, V, M, cap)
        # self-contained (Section 2.1, property 2): decoder rebuilds its own codebook
        back, cb2 = lzw.decode(codes, V, M, cap)
        assert back == x
        # replay equivalence: encoder-side and decoder-side codebooks are the same object
        assert cb2.entries == cb.entries
        # merge-size and capacity bounds
        assert all(2 <= len(e) <= max(M, 1) for e in cb.entries)
        if M == 1:
            assert cb.entries == [] and codes == x
        assert len(cb.entries) <= min(cap, max(len(codes) - 1, 0))
        assert -(-len(x) // M) <= len(codes) <= len(x)
        assert len(set(cb.entries)) == len(cb.entries)           # no duplicate phrases
        # entries_after is non-decreasing, grows by at most one per emitted code
        assert all(0 <= b - a <= 1 for a, b in zip([0] + after[:-1], after))
        # longest phrase of length k needs k(k-1)/2 + 1 tokens of input (the appendix's
        # O(sqrt N) bound with the constant that holds for LZW)
        k = max([len(e) for e in cb.entries], default=1)
        assert k * (k - 1) // 2 + 1 <= len(x)
        # every code refers to something that existed when it was emitted
        for i, z in enumerate(codes):
            assert z < V + (after[i - 1] if i else 0)
        assert lzw.base_token_count(cb, codes) == len(x)


def test_prefix_property_online():
    # online (Section 2.1, property 1): compressing a prefix gives a prefix of the codes,
    # except for the prefix's own final flush code
    V, x = _streams()[0]
    x = [int(t) for t in x[:200]]
    full, _, _ = lzw.encode(x, V, 3, 256)
    for k in range(1, len(x)):
        part, _, _ = lzw.encode(x[:k], V, 3, 256)
        assert part[:-1] == full[:len(part) - 1]


def _check_longest_match(x, V, M, cap):
    codes, after, cb = lzw.encode(x, V, M, cap)
    p = 0
    for i, z in enumerate(codes):
        n_before = after[i - 1] if i else 0
        ph = cb.phrase(z)
        assert tuple(x[p:p + len(ph)]) == ph
        # scan the WHOLE codebook as it stood: nothing longer may match here
        for e in cb.entries[:n_before]:
            if len(e) > len(ph):
                assert tuple(x[p:p + len(e)]) != e
        # the entry created by this emission is (phrase + next token) unless blocked
        if after[i] > n_before:
            assert cb.entries[n_before] == ph + (x[p + len(ph)],)
            assert len(ph) < M and n_before < cap
        elif p + len(ph) < len(x):
            cand = ph + (x[p + len(ph)],)
            assert len(ph) >= M or n_before >= cap or cand in cb.entries[:n_before]
        p += len(ph)
    assert p == len(x)
    back, _ = lzw.decode(codes, V, M, cap)
    assert back == list(x)


def test_brute_force_tiny_vocabularies():
    # unambiguous (Section 2.1, property 3): the parse is the greedy longest match, checked by
    # enumeration against a scan of the whole codebook
    for V, Tmax in ((2, 10), (3, 7)):
        for T in range(0, Tmax + 1):
            for x in itertools.product(range(V), repeat=T):
                for M in (2, 3):
                    for cap in (1, 4, 10 ** 6):
                        _check_longest_match(x, V, M, cap)


def test_step_rejects_nonexistent_hypertoken_and_keeps_state():
    cb = lzw.Codebook(6, 3, 256)
    cb.encode([0, 1, 2, 3, 0, 1])
    n, prev = cb.n(), cb.prev
    assert cb.step(6 + n + 1) == -1 and cb.status & lzw.BAD_TOKEN
    assert cb.n() == n and cb.prev == prev
    cb.status = 0
    assert cb.step(-1) == -1 and cb.status & lzw.BAD_TOKEN
    # special-case id is legal only when the step really creates it
    cb = lzw.Codebook(2, 3, 256)
    cb.step(0)
    assert cb.step(2) == 0 and cb.status == 0 and cb.phrase(2) == (0, 0)
    cb = lzw.Codebook(2, 3, 256)
    assert cb.step(2) == -1 and cb.status & lzw.BAD_TOKEN         # nothing precedes it
    cb = lzw.Codebook(2, 1, 256)
    cb.step(0)
    assert cb.step(2) == -1 and cb.status & lzw.BAD_TOKEN         # M forbids the entry


def test_step_does_not_duplicate_on_non_canonical_streams():
    # generation may emit "to","be" although "to be" exists: no second entry with that content
    cb = lzw.Codebook(6, 3, 256)
    cb.encode([0, 1, 2])                  # entries: (0,1) (1,2); prev = 2
    cb.step(0)                            # (2,0)
    assert cb.step(1) == -1               # candidate (0,1) exists already
    assert len(set(cb.entries)) == len(cb.entries)


def test_generator_compression_is_in_a_plausible_range():
    # context only: the paper's compression-rate table (merge-size ablation) reports 68-75 %
    # at M=2..5 on real text; the synthetic streams should be of that order, not degenerate
    w = si.WORKLOADS["phi3_mini_head"]
    x = si.token_stream(w.V, 2048, w.zipf_s, w.copy_p, w.seg_min, w.seg_max, 5)
    codes, _, _ = lzw.encode([int(t) for t in x], w.V, w.M, w.cap)
    assert 0.45 < len(codes) / len(x) < 0.98


def test_expand_with_resident_codebook_matches_self_contained_decode():
    """expand() reads the finished codebook, decode() rebuilds its own: both must give back the
    original tokens; a code past the end of the codebook stops the expansion before it."""
    for V, x in _streams():
        x = [int(t) for t in x]
        for M, cap in ((3, 100000), (4, 17), (2, 0)):
            codes, _, cb = lzw.encode(x, V, M, cap)
            toks, done = lzw.expand(cb, codes)
            assert toks == x and done == len(codes)
            back, _ = lzw.decode(codes, V, M, cap)
            assert back == toks
            if len(codes) >= 3:
                broken = list(codes)
                broken[2] = V + cb.n()                       # names no entry of the finished book
                t2, d2 = lzw.expand(cb, broken)
                assert d2 == 2 and t2 == x[:len(t2)]
                assert len(t2) == lzw.base_token_count(cb, codes[:2])


def test_lookup_of_base_tokens_is_a_row_gather_and_flags_missing_hypertokens():
    from oracle import embedding as oemb
    rng = np.random.default_rng(5)
    V, d, B, cap = 11, 8, 2, 4
    W = rng.standard_normal((V, d))
    E = rng.standard_normal((B, cap, d))
    codes = [3, 10, 0, 7]
    out, bad = oemb.lookup(codes, [0, 1, 1, 0], W, E, [0, 0])
    assert bad == [] and np.array_equal(out, np.take(W, codes, axis=0))
    out, bad = oemb.lookup([V + 1, V + 2, V], [0, 0, 1], W, E, [2, 3])
    assert bad == [0] and np.array_equal(out[0], E[0, 1]) and not out[1].any()
    assert np.array_equal(out[2], E[1, 0])
    # -1 is "no token" (a sequence that has finished): a zero row that is not an error; any
    # other id outside [0, V + n) is one
    out, bad = oemb.lookup([-1, 3, -2], [0, 1, 1], W, E, [2, 3])
    assert bad == [1] and not out[0].any() and np.array_equal(out[1], W[3]) and not out[2].any()


def test_lookup_of_a_hypertoken_under_the_averaging_encoder_is_the_mean_of_its_base_rows():
    """Ties the lookup to the codebook: with the parameter-free averaging hyper-encoder a
    hypertoken's cached row is the mean of W_E over the base tokens it decompresses to, so the
    lookup of the compressed stream, weighted by phrase lengths, sums to the lookup of the
    original stream."""
    from oracle import embedding as oemb
    from oracle import hyper_encoder as ohe
    rng = np.random.default_rng(6)
    V, d, M, cap = 7, 4, 3, 64
    x = [int(t) for t in rng.integers(0, V, size=200)]
    codes, _, cb = lzw.encode(x, V, M, cap)
    W = rng.standard_normal((V, d))
    pos0 = [np.zeros((M, d))]                               # no layers, zero positions: averaging
    E = np.zeros((1, cap, d))
    for k, e in enumerate(cb.entries):
        E[0, k] = ohe.hyper_embed_one(list(e), W, pos0, 1)
    rows, bad = oemb.lookup(codes, [0] * len(codes), W, E, [cb.n()])
    assert bad == []
    lens = np.array([len(cb.phrase(z)) for z in codes], dtype=np.float64)
    base_rows, _ = oemb.lookup(x, [0] * len(x), W, E, [cb.n()])
    np.testing.assert_allclose((rows * lens[:, None]).sum(0), base_rows.sum(0), rtol=0, atol=1e-9)
    # and one by one: each compressed row is the mean of its own slice of the base rows
    at = 0
    for r, z in enumerate(codes):
        L = int(lens[r])
        np.testing.assert_allclose(rows[r], base_rows[at:at + L].mean(0), rtol=0, atol=1e-12)
        at += L

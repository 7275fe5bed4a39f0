"""Pins for oracle/logits.py and oracle/decode_step.py (CPU only)."""
import numpy as np
import torch

from oracle import decode_step as ds, logits as lg
from paper_2506_01084_b200 import synth_inputs as si


def test_philox_known_answers():
    # test vectors published with the generator (Random123 known-answer file, philox4x32-10)
    kat = [((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
           ((0xffffffff,) * 4, (0xffffffff,) * 2,
            (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
           ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0),
            (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1))]
    for ctr, key, want in kat:
        got = lg.philox4x32_10(*[np.array([c]) for c in ctr], key[0], key[1])
        assert tuple(int(g[0]) for g in got) == want


def test_uniform_is_open_exact_in_fp32_and_counter_mapped():
    j = np.arange(4096)
    u = lg.uniform_open(j, row=3, step=(1 << 33) + 5, seed=(7 << 32) | 9)
    assert u.min() > 0.0 and u.max() < 1.0
    assert np.all(u.astype(np.float32).astype(np.float64) == u)
    # column j uses counter word j % 4 of block j // 4
    w = lg.philox4x32_10(np.array([10]), np.array([3]), np.array([5]), np.array([2]), 9, 7)
    for k in range(4):
        assert u[40 + k] == ((int(w[k][0]) >> 9) + 0.5) * 2.0 ** -23
    assert 0.45 < u.mean() < 0.55


def test_plain_definition_and_reductions():
    rng = np.random.default_rng(0)
    V, d, n = 300, 16, 37
    W = rng.normal(size=(V, d)); U = rng.normal(size=(n, d)); h = rng.normal(size=d)
    l = lg.joint_logits(h, W, U)
    assert l.shape == (V + n,)
    # no hypertokens: an ordinary LM head (library matmul, fp64)
    ref = (torch.from_numpy(h)[None] @ torch.from_numpy(W).T)[0].numpy()
    np.testing.assert_allclose(lg.joint_logits(h, W, None), ref, atol=1e-13)
    np.testing.assert_allclose(l[:V], ref, atol=1e-13)
    np.testing.assert_allclose(l[V:], [float(np.dot(U[i], h)) for i in range(n)], atol=1e-13)
    L = lg.lse(l)
    assert abs(np.exp(l - L).sum() - 1.0) < 1e-12                 # softmax normalises
    assert L >= lg.lse(l[:V])                                     # union >= static part
    np.testing.assert_allclose(L, float(torch.logsumexp(torch.from_numpy(l), 0)), atol=1e-12)
    # shift invariance and extreme magnitudes
    assert abs(lg.lse(l + 1000.0) - (L + 1000.0)) < 1e-9
    a, best, gap = lg.top2(l)
    assert best == l.max() and a == int(np.flatnonzero(l == l.max())[0])
    srt = np.sort(l)
    assert abs(gap - (srt[-1] - srt[-2])) < 1e-15
    # tie: lowest index wins, gap 0
    l2 = l.copy(); l2[5] = l2[200] = l.max() + 1.0
    a2, _, gap2 = lg.top2(l2)
    assert a2 == 5 and gap2 == 0.0


def test_gumbel_max_samples_from_softmax():
    rng = np.random.default_rng(1)
    l = rng.normal(size=6) * 1.5
    T = 0.7
    p = np.exp(l / T - lg.lse(l / T))
    counts = np.zeros(6)
    n = 20000
    for step in range(n):
        a, _, _ = lg.select(l, 1, T, seed=1234, step=step, row=0)
        counts[a] += 1
    # 5 sigma binomial bound per category
    assert np.all(np.abs(counts / n - p) < 5 * np.sqrt(p * (1 - p) / n) + 1e-3)
    # different rows / steps / seeds decorrelate
    g0 = lg.gumbel(np.arange(64), 0, 0, 1); g1 = lg.gumbel(np.arange(64), 1, 0, 1)
    g2 = lg.gumbel(np.arange(64), 0, 1, 1); g3 = lg.gumbel(np.arange(64), 0, 0, 2)
    assert len({g0.tobytes(), g1.tobytes(), g2.tobytes(), g3.tobytes()}) == 4


def test_round_to_storage_is_rne_bf16():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -3.1415926, 1e-30,
                  65504.0, 0.0])
    want = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(ds.round_to_storage(x, "bf16"), want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert ds.round_to_storage(np.array([1.0 + 2.0 ** -8]), "bf16")[0] == 1.0
    assert ds.round_to_storage(np.array([1.0 + 3 * 2.0 ** -8]), "bf16")[0] == 1.0 + 2.0 ** -6
    r = np.random.default_rng(2).normal(size=10000) * 3
    want = torch.tensor(r).float().bfloat16().double().numpy()
    np.testing.assert_array_equal(ds.round_to_storage(r, "bf16"), want)


def test_session_step_consistency_on_tiny_workload():
    w = si.WORKLOADS["tiny"].scaled(T=64, steps=8)
    toks = si.make_tokens(w, 1)
    W_E, W_U = si.make_tables(w, 1)
    encE = [t.double().numpy() for t in si.make_encoder(w, 2)]
    encU = [t.double().numpy() for t in si.make_encoder(w, 3)]
    s = ds.Session(w.V, w.M, w.cap, w.B, w.heads, w.dtype, W_E.double().numpy(),
                   W_U.double().numpy(), encE, encU)
    codes, after = s.prefill([toks[b].tolist() for b in range(w.B)])
    hid = si.make_hidden(w, w.steps * w.B, 1).double().numpy().reshape(w.steps, w.B, w.d)
    for t in range(w.steps):
        n0 = [bk.n() for bk in s.books]
        sc, new = s.step(hid[t], mode=0)
        for b in range(w.B):
            # both caches always cover exactly the codebook (consistent vocabulary updates)
            assert s.E_h[b].shape[0] == s.U_h[b].shape[0] == s.books[b].n()
            assert s.books[b].n() - n0[b] in (0, 1)               # at most one entry per step
            assert sc[b]["l"].shape[0] == w.V + n0[b]
            assert 0 <= sc[b]["choice"] < w.V + n0[b]


# ------------------------------------------------------------------------------------------------
# top-k / nucleus filtering (not defined by the paper; the usual definitions, ties kept together)
# ------------------------------------------------------------------------------------------------
def test_filter_mask_on_a_distribution_with_known_prefix_sums():
    p = np.array([0.05, 0.5, 0.15, 0.3])                      # descending order: columns 1, 3, 2, 0
    l = np.log(p)
    as_set = lambda m: set(np.nonzero(m)[0].tolist())
    assert as_set(lg.filter_mask(l, 1.0, 0, 0.49)) == {1}     # the first probability alone reaches 0.49
    assert as_set(lg.filter_mask(l, 1.0, 0, 0.51)) == {1, 3}
    assert as_set(lg.filter_mask(l, 1.0, 0, 0.79)) == {1, 3}
    assert as_set(lg.filter_mask(l, 1.0, 0, 0.81)) == {1, 3, 2}
    assert as_set(lg.filter_mask(l, 1.0, 0, 1.0)) == {0, 1, 2, 3}
    assert as_set(lg.filter_mask(l, 1.0, 2, 1.0)) == {1, 3}
    assert as_set(lg.filter_mask(l, 1.0, 3, 0.6)) == {1, 3}   # intersection of the two filters
    assert as_set(lg.filter_mask(l, 1.0, 1, 0.99)) == {1}
    # temperature reshapes the probabilities the nucleus is taken on: T = 0.5 squares them
    q = p ** 2 / (p ** 2).sum()                               # 0.0068, 0.68, 0.061, 0.245
    assert as_set(lg.filter_mask(l, 0.5, 0, 0.7)) == {1, 3} and q[1] < 0.7 < q[1] + q[3]
    # ties are kept together
    lt = np.array([1.0, 3.0, 3.0, 0.0, 3.0])
    assert as_set(lg.filter_mask(lt, 1.0, 1, 1.0)) == {1, 2, 4}
    assert as_set(lg.filter_mask(lt, 1.0, 0, 0.1)) == {1, 2, 4}


def test_select_filtered_special_cases_reduce_to_argmax_and_to_plain_sampling():
    rng = np.random.default_rng(8)
    for t in range(20):
        l = rng.standard_normal(200) * 2.0
        a, keep, _ = lg.select_filtered(l, 0.8, 1, 1.0, 77, t, 3)
        assert a == int(np.argmax(l)) and keep.sum() == 1       # k = 1: the argmax, whatever the noise
        a2, keep2, _ = lg.select_filtered(l, 0.8, 0, 1.0, 77, t, 3)
        assert keep2.all() and a2 == lg.select(l, 1, 0.8, 77, t, 3)[0]   # no filter: plain Gumbel-max
        a3, keep3, _ = lg.select_filtered(l, 0.8, 7, 0.9, 77, t, 3)
        assert keep3[a3] and keep3[int(np.argmax(l))] and keep3.sum() <= 7
        pr = np.exp((l - l.max()) / 0.8); pr /= pr.sum()
        kp = lg.filter_mask(l, 0.8, 0, 0.9)
        assert pr[kp].sum() >= 0.9 and pr[kp].sum() - pr[kp].min() < 0.9   # the shortest such prefix


def test_select_filtered_frequencies_follow_the_renormalised_distribution():
    l = np.log(np.array([0.4, 0.25, 0.2, 0.1, 0.05]))
    counts = np.zeros(5)
    n = 6000
    for t in range(n):
        a, keep, _ = lg.select_filtered(l, 1.0, 3, 1.0, 5, t, 0)
        counts[a] += 1
    want = np.array([0.4, 0.25, 0.2, 0.0, 0.0]) / 0.85
    assert counts[3] == 0 and counts[4] == 0
    assert np.abs(counts / n - want).max() < 0.02

"""GPU parity of top-k / nucleus filtered sampling against the CPU oracle.  Both sides get the
same fp32 logits (the kernel is a function of stored logits), so the kept SET is compared exactly
wherever floating-point summation cannot move the nucleus boundary, and the sample exactly unless
the oracle's two best perturbed scores are closer than the usual gap."""
import numpy as np
import pytest
import torch

from oracle import logits as olg
from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import synth_inputs as si
from tests._harness import GAP

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _band(l, T, top_p, delta=2e-5):
    """Columns whose cumulative probability (descending order) lies within delta of top_p: fp32
    summation of the masses may put the nucleus boundary anywhere among them."""
    if top_p >= 1.0:
        return np.zeros(l.shape[0], dtype=bool)
    order = np.argsort(-l, kind="stable")
    pr = np.exp((l[order] - l[order[0]]) / T)
    cum = np.cumsum(pr) / pr.sum()
    near = np.zeros(l.shape[0], dtype=bool)
    near[order[np.abs(cum - top_p) <= delta]] = True
    # ... together with everything tied with one of them
    vals = np.unique(l[near])
    return near | np.isin(l, vals)


def _run(l32, n_cols, top_k, top_p, T, seed, step, row_base=0):
    N = l32.shape[0]
    g = torch.from_numpy(l32).to(DEV)
    choice = torch.full((N,), -7, dtype=torch.int32, device=DEV)
    kept = torch.full((N,), -7, dtype=torch.int32, device=DEV)
    zb.z2z_sample_filtered(g, torch.tensor(n_cols, dtype=torch.int32, device=DEV), top_k, top_p, T, seed, step,
                           choice, kept, row_base)
    return choice.cpu().numpy(), kept.cpu().numpy()


@pytest.mark.parametrize("top_k,top_p,T", [(0, 1.0, 1.0), (1, 1.0, 0.7), (50, 1.0, 1.0), (0, 0.9, 1.0), (0, 0.3, 0.5),
                                           (40, 0.95, 0.8), (7, 0.999, 1.3), (100000, 0.5, 1.0)])
def test_filtered_sampling_matches_oracle(top_k, top_p, T):
    rng = np.random.default_rng(3)
    N, C = 6, 37000                                            # a phi3-sized joint vocabulary, ragged rows
    l32 = (rng.standard_normal((N, C)) * 2.5).astype(np.float32)
    l32[1, :200] = l32[1, 0]                                    # a plateau of ties, also at the very top
    l32[2, 5000:5100] = l32[2].max()
    n_cols = [C, C - 1, 32064, 1000, 1, C - 4097]
    checked = exact = 0
    for step in range(3):
        got, kept = _run(l32, n_cols, top_k, top_p, T, 99, step, row_base=11)
        for r in range(N):
            l = l32[r, :n_cols[r]].astype(np.float64)
            a, keep, gap = olg.select_filtered(l, T, top_k, top_p, 99, step, 11 + r)
            band = _band(l, T, top_p)                          # where fp32 summation may move the boundary
            slack = int(band.sum())
            assert abs(int(kept[r]) - int(keep.sum())) <= slack, (r, kept[r], int(keep.sum()), slack)
            assert 0 <= got[r] < n_cols[r] and (keep[got[r]] or band[got[r]])
            if got[r] != a:
                assert gap < GAP or band[got[r]] or band[a], (r, step, got[r], a, gap)
            exact += int(slack == 0)
            checked += 1
    assert checked == 18 and exact >= (18 if top_p >= 1.0 else 0)


@pytest.mark.parametrize("C", [37001, 4099, 5])
def test_filtered_sampling_rows_that_start_off_a_16_byte_boundary(C):
    # an odd row stride: rows 1.. take the scalar loads; rows whose length is no multiple of four
    # take the ragged tail of the vector loads
    rng = np.random.default_rng(13)
    N = 4
    l32 = (rng.standard_normal((N, C)) * 2.0).astype(np.float32)
    n_cols = [C, C - 1, max(C - 2, 1), max(C - 3, 1)]
    for top_k, top_p in ((9, 1.0), (0, 0.8), (1, 1.0)):
        got, kept = _run(l32, n_cols, top_k, top_p, 0.9, 5, 2)
        for r in range(N):
            l = l32[r, :n_cols[r]].astype(np.float64)
            a, keep, gap = olg.select_filtered(l, 0.9, top_k, top_p, 5, 2, r)
            band = _band(l, 0.9, top_p)
            assert abs(int(kept[r]) - int(keep.sum())) <= int(band.sum())
            assert keep[got[r]] or band[got[r]]
            if got[r] != a:
                assert gap < GAP or band[got[r]] or band[a]


@pytest.mark.parametrize("N", [20, 40, 80])
def test_filtered_sampling_with_every_cluster_size(N):
    # the rows of a batch share the SMs: 20, 40 and 80 rows are worked on by clusters of 4, 2 and
    # 1 CTAs per row (up to 9 rows by clusters of 8, as in the tests above)
    rng = np.random.default_rng(17 + N)
    C = 9001
    l32 = (rng.standard_normal((N, C)) * 2.0).astype(np.float32)
    n_cols = [C - (r % 7) for r in range(N)]
    got, kept = _run(l32, n_cols, 30, 0.9, 1.1, 21, 4, row_base=3)
    for r in range(N):
        l = l32[r, :n_cols[r]].astype(np.float64)
        a, keep, gap = olg.select_filtered(l, 1.1, 30, 0.9, 21, 4, 3 + r)
        band = _band(l, 1.1, 0.9)
        assert abs(int(kept[r]) - int(keep.sum())) <= int(band.sum())
        assert keep[got[r]] or band[got[r]]
        if got[r] != a:
            assert gap < GAP or band[got[r]] or band[a]


def test_filtered_sampling_small_rows_and_frequencies():
    # tiny rows, exhaustively comparable; and frequencies over many steps against the renormalised distribution
    p = np.array([0.4, 0.25, 0.2, 0.1, 0.05])
    l32 = np.log(p).astype(np.float32)[None, :].repeat(2, 0)
    counts = np.zeros(5)
    n = 1500
    for step in range(n):
        got, kept = _run(l32, [5, 3], 3, 1.0, 1.0, 5, step)
        assert kept.tolist() == [3, 3]
        a, _, gap = olg.select_filtered(l32[0].astype(np.float64), 1.0, 3, 1.0, 5, step, 0)
        assert got[0] == a or gap < GAP
        counts[got[0]] += 1
    want = np.array([0.4, 0.25, 0.2, 0.0, 0.0]) / 0.85
    assert counts[3] == 0 and counts[4] == 0 and np.abs(counts / n - want).max() < 0.04


def test_filtered_sampling_on_logits_stored_by_the_logits_kernel():
    """End of the chain: joint logits of a decode batch stored by z2z_dynamic_logits, then filtered
    sampling on them; the oracle filters ITS OWN fp64 logits, so a row is compared where the top-k
    boundary has a margin."""
    w = si.Workload("filt", V=3000, d=256, dtype="bf16", B=4, T=120, M=3, cap=64, zipf_s=1.1, copy_p=0.4, seg_min=3,
                    seg_max=10, steps=1, enc_layers=0, enc_heads=2, enc_dff=512)
    cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, 0, 1, 8)
    cb = zb.Codebook(cfg, DEV)
    tokens = si.make_tokens(w, 9)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=DEV)
    clen = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    zb.z2z_lzw_encode(cb, torch.from_numpy(tokens).to(DEV), None, codes, clen, None)
    _, n = zb.z2z_status(cb)
    _, W_U = si.make_tables(w, 9)
    U_h = si.normal_tensor((w.B, w.cap, w.d), 0.05, 10, torch.bfloat16)
    hid = si.make_hidden(w, w.B, 11)
    ld = w.V + w.cap
    dbg = torch.zeros(w.B, ld, dtype=torch.float32, device=DEV)
    lse = torch.zeros(w.B, dtype=torch.float32, device=DEV)
    am = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    mxl = torch.zeros(w.B, dtype=torch.float32, device=DEV)
    zb.z2z_dynamic_logits(cb, hid.to(DEV), None, None, W_U.to(DEV), U_h.to(DEV), zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                          lse, am, mxl, logits_debug=dbg)
    n_cols = [w.V + int(n[b]) for b in range(w.B)]
    choice = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    kept = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    zb.z2z_sample_filtered(dbg, torch.tensor(n_cols, dtype=torch.int32, device=DEV), 20, 1.0, 0.8, 7, 3, choice, kept)
    got, k = choice.cpu().numpy(), kept.cpu().numpy()
    compared = 0
    for b in range(w.B):
        l = olg.joint_logits(hid[b].double().numpy(), W_U.double().numpy(), U_h[b, :int(n[b])].double().numpy())
        a, keep, gap = olg.select_filtered(l, 0.8, 20, 1.0, 7, 3, b)
        assert 0 <= got[b] < n_cols[b]
        ls = np.sort(l)[::-1]
        if ls[19] - ls[20] > 1e-4:                                # the 20th and 21st logit are well apart
            assert k[b] == int(keep.sum()) == 20
            assert keep[got[b]]
            assert got[b] == a or gap < GAP
            compared += 1
    assert compared >= 2

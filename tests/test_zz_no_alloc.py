"""The entry point for callers that cannot allocate device memory (z2z_logits_static_scratch),
checked through the C ABI against the ordinary z2z_dynamic_logits on the same inputs and, row by
row, against the fp64 oracle.

Such callers (a plug-in in a process that handed out all device memory at start-up, code that
must not enter an allocator) pass inputs and outputs only; the kernel's partial reductions live
in a fixed array inside the library that every call shares and that keeps the previous call's
contents.  So the check runs two different calls in a row: stale partials of the first must not
leak into the second.  This file sorts last on purpose, so that a run stopping at the first
failure has already run everything else."""
import numpy as np
import pytest
import torch

from oracle import logits as olg, lzw as olzw
from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import synth_inputs as si
from tests._harness import GAP, TOL, f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

W = si.Workload("noalloc_bf16", V=1000, d=256, dtype="bf16", B=3, T=160, M=4, cap=96,
                zipf_s=1.1, copy_p=0.4, seg_min=3, seg_max=12, steps=0, enc_layers=0,
                enc_heads=2, enc_dff=512)


@pytest.mark.parametrize("w", [W, W.scaled(name="noalloc_fp32", dtype="fp32", d=72)],
                         ids=lambda w: w.name)
def test_static_scratch_matches_ordinary_entry_point_twice(w):
    cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, 0, 1, 8)
    cb = zb.Codebook(cfg, DEV)
    tokens = si.make_tokens(w, 41)
    tok = torch.from_numpy(tokens).to(DEV)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=DEV)
    clen = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    zb.z2z_lzw_encode(cb, tok, None, codes, clen, None)        # gives each sequence its own n_b
    _, n = zb.z2z_status(cb)
    assert int(n.sum()) > 0
    n_oracle = [olzw.encode(tokens[b].tolist(), w.V, w.M, w.cap)[2].n() for b in range(w.B)]
    assert n.tolist() == n_oracle                               # the oracle side below uses its own counts
    n_dev = n.to(DEV)
    W_U = si.make_tables(w, 41)[1].to(DEV)
    U_h = si.normal_tensor((w.B, w.cap, w.d), 0.05, 43, w.torch_dtype).to(DEV)
    for call, rows_per_seq in enumerate(([40, 3, 70], [1, 90, 0])):
        row_seq = torch.tensor([b for b in range(w.B) for _ in range(rows_per_seq[b])],
                               dtype=torch.int32, device=DEV)
        N = row_seq.numel()
        hid = si.make_hidden(w, N, 50 + call).to(DEV)
        ref = {k: torch.zeros(N, dtype=torch.float32, device=DEV) for k in ("lse", "max")}
        ref_am = torch.zeros(N, dtype=torch.int32, device=DEV)
        zb.z2z_dynamic_logits(cb, hid, row_seq, None, W_U, U_h, zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                              ref["lse"], ref_am, ref["max"])
        got = {k: torch.full((N,), float("nan"), dtype=torch.float32, device=DEV)
               for k in ("lse", "max")}
        got_am = torch.full((N,), -5, dtype=torch.int32, device=DEV)
        zb.z2z_logits_static_scratch(hid, row_seq, n_dev, W_U, U_h, w.cap, got["lse"], got_am,
                                     got["max"])
        torch.cuda.synchronize()
        # against the ordinary entry point: same reductions within the tolerance; a different index
        # only where the two maxima are a tie within the selection gap
        for k in ("lse", "max"):
            err = (got[k] - ref[k]).abs().max().item()
            assert err <= TOL, (call, k, err)
        differ = (got_am != ref_am).cpu().numpy()
        assert np.all((got["max"] - ref["max"]).abs().cpu().numpy()[differ] <= GAP)
        # against the oracle (Section 2.3 steps 7-9, the plain definition in fp64), every row
        H, WU64, U64 = f64(hid), f64(W_U), f64(U_h)
        g_lse, g_max, g_am = (x.cpu().numpy() for x in (got["lse"], got["max"], got_am))
        rs, nn = row_seq.cpu().numpy(), n_oracle
        for r in range(N):
            b = int(rs[r])
            l = olg.joint_logits(H[r], WU64, U64[b, :int(nn[b])])
            assert abs(g_lse[r] - olg.lse(l)) <= TOL, (call, r, g_lse[r], olg.lse(l))
            a, best, gap = olg.top2(l)
            assert abs(g_max[r] - best) <= TOL, (call, r)
            assert 0 <= g_am[r] < w.V + int(nn[b])
            if g_am[r] != a:
                assert gap < GAP and l[g_am[r]] >= best - GAP, (call, r, g_am[r], a, gap)


def test_static_scratch_ignores_counts_beyond_the_cache_rows():
    # d_n_hyper comes from the caller here (the ordinary entry point owns its counters): a count
    # above cap must not make the kernel read past a sequence's cap rows into its neighbour's
    w = W
    W_U = si.make_tables(w, 45)[1].to(DEV)
    U_h = si.normal_tensor((w.B, w.cap, w.d), 0.05, 46, w.torch_dtype).to(DEV)
    hid = si.make_hidden(w, w.B, 47).to(DEV)
    outs = []
    for counts in ([w.cap, w.cap, w.cap], [w.cap + 40, w.cap + 1, 65535]):
        n_dev = torch.tensor(counts, dtype=torch.int32, device=DEV)
        lse = torch.zeros(w.B, dtype=torch.float32, device=DEV)
        am = torch.zeros(w.B, dtype=torch.int32, device=DEV)
        mx = torch.zeros(w.B, dtype=torch.float32, device=DEV)
        zb.z2z_logits_static_scratch(hid, None, n_dev, W_U, U_h, w.cap, lse, am, mx)
        torch.cuda.synchronize()
        outs.append((lse.cpu(), am.cpu(), mx.cpu()))
    for x, y in zip(*outs):
        assert torch.equal(x, y)
    H, WU64, U64 = f64(hid), f64(W_U), f64(U_h)
    for b in range(w.B):
        l = olg.joint_logits(H[b], WU64, U64[b])
        assert abs(outs[1][0][b].item() - olg.lse(l)) <= TOL


def test_static_scratch_rejects_sizes_beyond_its_array():
    w = W
    n_dev = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    W_U = torch.zeros(w.V, w.d, dtype=torch.bfloat16, device=DEV)
    hid = torch.zeros(1025, w.d, dtype=torch.bfloat16, device=DEV)
    row_seq = torch.zeros(1025, dtype=torch.int32, device=DEV)
    with pytest.raises(zb.Z2ZError, match="1024 rows"):
        zb.z2z_logits_static_scratch(hid, row_seq, n_dev, W_U, None, 0, None, None, None)

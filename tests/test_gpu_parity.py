"""GPU parity: the CUDA path (through the C ABI binding) against the CPU oracle, element by
element, on the same seeded inputs.  Integer results are bit-exact; floats within the stated
tolerance; selections follow the oracle except inside its top-2 gap."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import embedding as oemb, lzw as olzw, logits as olg
from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import synth_inputs as si
from tests._harness import GAP, TOL, Pair, f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


# ------------------------------------------------------------------------------------------------
# LZW: bit-exact
# ------------------------------------------------------------------------------------------------
class LzwOnly:
    def __init__(self, V, M, cap, B):
        self.V, self.M, self.cap, self.B = V, M, cap, B
        self.cfg = zb.make_config(V, 8, M, cap, B, "fp32", 0, 1, 8)
        self.cb = zb.Codebook(self.cfg, DEV)

    def encode(self, tokens, lens=None):
        B, T = tokens.shape
        g_tok = torch.from_numpy(np.ascontiguousarray(tokens.astype(np.int32))).to(DEV)
        g_lens = None if lens is None else torch.tensor(lens, dtype=torch.int32, device=DEV)
        codes = torch.full((B, max(T, 1)), -7, dtype=torch.int32, device=DEV)
        after = torch.full((B, max(T, 1)), -7, dtype=torch.int32, device=DEV)
        clen = torch.zeros(B, dtype=torch.int32, device=DEV)
        zb.z2z_lzw_encode(self.cb, g_tok, g_lens, codes, clen, after)
        return codes.cpu().numpy(), clen.cpu().numpy(), after.cpu().numpy()

    def entries(self, b):
        cons, ln = zb.z2z_codebook_read(self.cb, b)
        st, n = zb.z2z_status(self.cb)
        return [tuple(int(x) for x in cons[k, :int(ln[k])]) for k in range(int(n[b]))], int(st[b])


def _compare_encode(V, M, cap, tokens, lens=None):
    B, T = tokens.shape
    g = LzwOnly(V, M, cap, B)
    codes, clen, after = g.encode(tokens, lens)
    for b in range(B):
        L = T if lens is None else lens[b]
        want, waft, ob = olzw.encode(tokens[b, :L].tolist(), V, M, cap)
        assert clen[b] == len(want)
        assert codes[b, :clen[b]].tolist() == want
        assert after[b, :clen[b]].tolist() == waft
        ents, st = g.entries(b)
        assert ents == ob.entries
        assert st & ~zb.ST_CAP_FROZEN == 0
        assert bool(st & zb.ST_CAP_FROZEN) == (len(ents) >= cap > 0)
    return g


def test_lzw_worked_example():
    path = os.path.join(os.path.dirname(__file__), "golden", "fig1_to_be_or_not_to_be.txt")
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, toks, codes, ents = [p.strip() for p in line.split("|")]
        V, M, cap = map(int, head.split())
        x = np.array([[int(t) for t in toks.split()]], dtype=np.int32)
        g = LzwOnly(V, M, cap, 1)
        got, clen, _ = g.encode(x)
        assert got[0, :clen[0]].tolist() == [int(c) for c in codes.split()]
        want_entries = [tuple(int(t) for t in e.split(":")[1].split(",")) for e in ents.split()]
        assert g.entries(0)[0] == want_entries


@pytest.mark.parametrize("name,T", [("tiny", None), ("phi3_mini_head", None),
                                    ("llama3_8b_head", None), ("prefill_heavy", None),
                                    ("long_context", None)])
def test_lzw_encode_full_configs(name, T):
    w = si.WORKLOADS[name]
    tokens = si.make_tokens(w, 17)
    _compare_encode(w.V, w.M, w.cap, tokens)


def test_lzw_encode_ragged_empty_and_freeze():
    w = si.WORKLOADS["tiny"].scaled(B=7, T=300)
    tokens = si.make_tokens(w, 3)
    lens = [0, 1, 2, 31, 32, 33, 300]
    _compare_encode(w.V, 3, 256, tokens, lens)
    _compare_encode(w.V, 3, 5, tokens, lens)          # freezes early
    _compare_encode(w.V, 1, 256, tokens, lens)        # M = 1: identity coding
    _compare_encode(w.V, 8, 256, tokens, lens)        # largest supported merge size
    _compare_encode(w.V, 3, 0, tokens, lens)          # no hypertokens at all
    rep = np.zeros((2, 500), dtype=np.int32); rep[1] = np.arange(500) % 3
    _compare_encode(5, 8, 1000, rep)                  # heavy self-overlap (special-case ids)


def test_lzw_brute_force_against_oracle():
    for V, Tmax in ((2, 10), (3, 7)):
        for T in range(1, Tmax + 1):
            allx = np.array(list(itertools.product(range(V), repeat=T)), dtype=np.int32)
            for s in range(0, len(allx), 1024):
                chunk = allx[s:s + 1024]
                for M in (2, 3):
                    for cap in (1, 4, 64):
                        _compare_encode(V, M, cap, chunk)


def test_lzw_step_replay_equals_encode_and_rejects_bad_ids():
    w = si.WORKLOADS["tiny"].scaled(B=5, T=200)
    tokens = si.make_tokens(w, 9)
    enc = [olzw.encode(tokens[b].tolist(), w.V, w.M, w.cap) for b in range(w.B)]
    g = LzwOnly(w.V, w.M, w.cap, w.B)
    steps = max(len(e[0]) for e in enc)
    new_entry = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    replay = [olzw.Codebook(w.V, w.M, w.cap) for _ in range(w.B)]
    for t in range(steps):
        act = [1 if t < len(enc[b][0]) else 0 for b in range(w.B)]
        z = [enc[b][0][t] if act[b] else 0 for b in range(w.B)]
        zb.z2z_lzw_step(g.cb, torch.tensor(z, dtype=torch.int32, device=DEV),
                        torch.tensor(act, dtype=torch.uint8, device=DEV), new_entry)
        got = new_entry.cpu().tolist()
        for b in range(w.B):
            want = replay[b].step(z[b]) if act[b] else -1
            assert got[b] == want
    for b in range(w.B):
        ents, st = g.entries(b)
        assert ents == enc[b][2].entries and st == 0
    # ids that name nothing: state untouched, BAD_TOKEN raised (consistent vocabulary updates)
    st0, n0 = zb.z2z_status(g.cb)
    bad = [w.V + int(n0[b]) + 1 for b in range(w.B)]
    bad[1] = -3
    zb.z2z_lzw_step(g.cb, torch.tensor(bad, dtype=torch.int32, device=DEV), None, new_entry)
    st1, n1 = zb.z2z_status(g.cb)
    assert torch.equal(n0, n1) and all(int(s) & zb.ST_BAD_TOKEN for s in st1)
    assert new_entry.cpu().tolist() == [-1] * w.B
    for b in range(w.B):
        assert g.entries(b)[0] == enc[b][2].entries
    # and the next legal code behaves as if the bad one had never been sent
    z = [int(tokens[b, 0]) for b in range(w.B)]
    zb.z2z_lzw_step(g.cb, torch.tensor(z, dtype=torch.int32, device=DEV), None, new_entry)
    for b in range(w.B):
        assert new_entry.cpu().tolist()[b] == replay[b].step(z[b])


def test_lzw_step_special_case_id():
    g = LzwOnly(2, 3, 16, 1)
    ne = torch.zeros(1, dtype=torch.int32, device=DEV)
    ob = olzw.Codebook(2, 3, 16)
    for z in [0, 2, 3, 0, 4]:      # 2 and 3 are created by the step that receives them
        zb.z2z_lzw_step(g.cb, torch.tensor([z], dtype=torch.int32, device=DEV), None, ne)
        assert ne.item() == ob.step(z)
        ents, st = g.entries(0)
        assert ents == ob.entries and st == ob.status


# ------------------------------------------------------------------------------------------------
# Hyper-encoder
# ------------------------------------------------------------------------------------------------
SMALL_BF16 = si.Workload("small_bf16", V=1000, d=256, dtype="bf16", B=3, T=160, M=4, cap=96,
                         zipf_s=1.1, copy_p=0.4, seg_min=3, seg_max=12, steps=12, enc_layers=2,
                         enc_heads=2, enc_dff=512)
SMALL_FP32 = SMALL_BF16.scaled(name="small_fp32", dtype="fp32", d=72, enc_heads=3, enc_dff=200,
                               M=5)


def _prefill_both(p: Pair):
    w = p.w
    codes, clen, after = p.gpu_encode()
    ocodes, oafter = p.oracle.prefill([p.tokens[b].tolist() for b in range(w.B)])
    for b in range(w.B):
        assert codes[b, :clen[b]].tolist() == ocodes[b]
        assert after[b, :clen[b]].tolist() == oafter[b]
    p.check_codebooks()
    total = sum(bk.n() for bk in p.oracle.books)
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, total, p.E_h, p.E_f32)
    if not w.tied:
        zb.z2z_hyper_embed(p.cb, zb.CACHE_UNEMBED, p.g_WU, p.g_encU, None, None, total, p.U_h,
                           p.U_f32)
    worst = 0.0
    for b in range(w.B):
        worst = max(worst, p.check_cache_rows(b, 0, p.oracle.books[b].n()))
    return ocodes, worst


@pytest.mark.parametrize("w", [si.WORKLOADS["tiny"], SMALL_BF16, SMALL_FP32,
                               SMALL_BF16.scaled(name="avg", enc_layers=0),
                               SMALL_BF16.scaled(name="one_layer", enc_layers=1),
                               SMALL_BF16.scaled(name="attn_only", enc_layers=1, enc_ffn=0),
                               SMALL_FP32.scaled(name="attn_only_fp32", enc_layers=2, enc_ffn=0),
                               SMALL_BF16.scaled(name="tied", tied=1)],
                         ids=lambda w: w.name)
def test_hyper_embed_all_prefill_entries(w):
    p = Pair(w, seed=5)
    _, worst = _prefill_both(p)
    print(f"{w.name}: max |hyper-embedding error| = {worst:.3e}")
    # rows beyond n_b were not touched
    for b in range(w.B):
        n = p.oracle.books[b].n()
        assert float(p.E_h[b, n:].abs().max().item() if n < w.cap else 0.0) == 0.0
    if w.dtype == "fp32":
        for b in range(w.B):
            assert p.check_cache_rows(b, 0, p.oracle.books[b].n(), tol=2e-5) <= 2e-5


def test_hyper_embed_explicit_ranges_and_incremental():
    w = SMALL_BF16
    p = Pair(w, seed=6)
    p.gpu_encode()
    p.oracle.prefill([p.tokens[b].tolist() for b in range(w.B)])
    n = [bk.n() for bk in p.oracle.books]
    first = [0, min(5, n[1]), n[2]]
    count = [min(3, n[0]), max(0, n[1] - 5), 0]
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE,
                       torch.tensor(first, dtype=torch.int32, device=DEV),
                       torch.tensor(count, dtype=torch.int32, device=DEV), sum(count), p.E_h, p.E_f32)
    got = p.E_f32.cpu().double().numpy()
    for b in range(w.B):
        lo, hi = first[b], first[b] + count[b]
        if hi > lo:
            assert np.abs(got[b, lo:hi] - p.oracle.E_exact[b][lo:hi]).max() <= TOL
        assert np.all(got[b, :lo] == 0) and np.all(got[b, hi:] == 0)
    # the same ranges with the exact pass count (max_entries < 0): the same rows, nothing else touched
    ranges_run = p.E_f32.clone()
    p.E_f32.zero_()
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE,
                       torch.tensor(first, dtype=torch.int32, device=DEV),
                       torch.tensor(count, dtype=torch.int32, device=DEV), -1, p.E_h, p.E_f32)
    assert float((p.E_f32 - ranges_run).abs().max()) <= 1e-5
    # NULL ranges after that: "everything since the last NULL call" = all entries
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, 0, p.E_h, p.E_f32)
    got = p.E_f32.cpu().double().numpy()
    for b in range(w.B):
        assert np.abs(got[b, :n[b]] - p.oracle.E_exact[b]).max() <= TOL
    # max_entries < 0: the call reads the entry count back and launches only passes with work;
    # the same rows come out, and a call with nothing to do launches no encoder kernel at all
    first_run = p.E_f32.clone()
    zb.z2z_codebook_init(p.cb)
    p.gpu_encode()
    p.E_f32.zero_()
    zb.z2z_profile_read(p.cb)
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, -1, p.E_h, p.E_f32)
    assert float((p.E_f32 - first_run).abs().max()) <= 1e-5
    _, launches = zb.z2z_profile_read(p.cb)
    assert launches["encoder_gemm"] > 0
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, -1, p.E_h, p.E_f32)   # nothing new
    _, launches = zb.z2z_profile_read(p.cb)
    assert launches["encoder_gemm"] == 0
    assert float((p.E_f32 - first_run).abs().max()) <= 1e-5


# ------------------------------------------------------------------------------------------------
# Joint logits and reductions
# ------------------------------------------------------------------------------------------------
def _logits_case(w, seed, rows_per_seq, causal, select, temperature=0.8, tensor_cores=True,
                 debug=True):
    p = Pair(w, seed=seed, generic_encoder=False, tensor_cores=tensor_cores)
    codes, clen, after = p.gpu_encode()
    ocodes, oafter = p.oracle.prefill([p.tokens[b].tolist() for b in range(w.B)])
    n = [bk.n() for bk in p.oracle.books]
    # synthetic hyper-unembedding rows straight from the generator (same values on both sides)
    U = si.normal_tensor((w.B, max(w.cap, 1), w.d), 0.05, seed + 100, w.torch_dtype)
    p.U_h.copy_(U.to(p.dev))
    U64 = f64(U)
    rng = np.random.default_rng(seed)
    row_seq, row_nvis = [], []
    for b in range(w.B):
        for _ in range(rows_per_seq[b]):
            row_seq.append(b)
            row_nvis.append(int(rng.integers(0, n[b] + 1)) if causal else n[b])
    N = len(row_seq)
    hid = si.make_hidden(w, N, seed)
    targets = [int(rng.integers(0, w.V + w.cap)) for _ in range(N)]
    g_hid = hid.to(p.dev)
    out = {k: torch.zeros(N, dtype=torch.float32, device=p.dev) for k in ("lse", "max", "tl")}
    am = torch.zeros(N, dtype=torch.int32, device=p.dev)
    smp = torch.zeros(N, dtype=torch.int32, device=p.dev)
    dbg = torch.full((N, w.V + w.cap), float("nan"), dtype=torch.float32, device=p.dev)
    zb.z2z_dynamic_logits(p.cb, g_hid, torch.tensor(row_seq, dtype=torch.int32, device=p.dev),
                          torch.tensor(row_nvis, dtype=torch.int32, device=p.dev) if causal else None,
                          p.g_WU, p.U_h, select, temperature, 0xABCDEF12345, 77,
                          torch.tensor(targets, dtype=torch.int32, device=p.dev) if debug else None,
                          out["lse"], am, out["max"], smp if select else None,
                          out["tl"] if debug else None, dbg if debug else None)
    dbg = dbg.cpu().double().numpy()
    lse, mx, tl = (out[k].cpu().double().numpy() for k in ("lse", "max", "tl"))
    am, smp = am.cpu().numpy(), smp.cpu().numpy()
    H = f64(hid)
    worst = 0.0
    for r in range(N):
        b, nv = row_seq[r], row_nvis[r]
        l = olg.joint_logits(H[r], p.oracle.W_U, U64[b, :nv])
        if debug:
            got = dbg[r, :w.V + nv]
            err = np.abs(got - l).max()
            worst = max(worst, err)
            assert err <= TOL
            assert np.all(np.isnan(dbg[r, w.V + nv:]))        # invisible columns never computed
        assert abs(lse[r] - olg.lse(l)) <= TOL, (r, lse[r], olg.lse(l))
        worst = max(worst, abs(lse[r] - olg.lse(l)))
        a, best, gap = olg.top2(l)
        assert abs(mx[r] - best) <= TOL
        if am[r] != a:
            assert gap < GAP and l[am[r]] >= best - GAP
        if debug:
            if targets[r] < w.V + nv:
                assert abs(tl[r] - l[targets[r]]) <= TOL
            else:
                assert np.isnan(tl[r])
        if select:
            ch, scores, sgap = olg.select(l, 1, temperature, 0xABCDEF12345, 77, r)
            if smp[r] != ch:
                assert sgap < GAP and scores[smp[r]] >= scores[ch] - GAP
    return worst


@pytest.mark.parametrize("w", [si.WORKLOADS["tiny"].scaled(B=2), SMALL_BF16, SMALL_FP32],
                         ids=lambda w: w.name)
@pytest.mark.parametrize("causal,select", [(False, 0), (True, 1)])
def test_dynamic_logits_elementwise(w, causal, select):
    rows = [1] * w.B if not causal else [70, 0, 5][:w.B] + [3] * max(0, w.B - 3)
    worst = _logits_case(w, 11, rows, causal, select)
    print(f"{w.name}: max |logit error| = {worst:.3e}")


def test_dynamic_logits_no_hypertokens_is_plain_lm_head():
    w = SMALL_BF16.scaled(cap=0, name="nocap")
    worst = _logits_case(w, 12, [2, 1, 1], False, 0)
    assert worst <= TOL


# ------------------------------------------------------------------------------------------------
# Whole decode step, following the GPU's selections inside the oracle's top-2 gap
# ------------------------------------------------------------------------------------------------
def _decode_follow(w, seed, select, steps=None, forced_every=0, tensor_cores=True, host_results=False,
                   sits_out=None):
    p = Pair(w, seed=seed, tensor_cores=tensor_cores)
    _prefill_both(p)
    for b in range(w.B):
        p.force_caches_from_oracle(b, 0, p.oracle.books[b].n())
    steps = w.steps if steps is None else steps
    hid = si.make_hidden(w, steps * w.B, seed + 1).view(steps, w.B, w.d)
    H = f64(hid)
    g_hid = hid.to(p.dev)
    nxt = torch.zeros(w.B, dtype=torch.int32, device=p.dev)
    sel = torch.zeros(w.B, dtype=torch.int32, device=p.dev)
    lse = torch.zeros(w.B, dtype=torch.float32, device=p.dev)
    new = torch.zeros(w.B, dtype=torch.int32, device=p.dev)
    if host_results:          # pinned host memory, mapped into the device's address space
        nxt, sel, lse, new = (x.cpu().pin_memory() for x in (nxt, sel, lse, new))
    nxt_emb = torch.zeros(w.B, w.d, dtype=w.torch_dtype, device=p.dev)
    followed = 0
    worst_lse = 0.0
    rng = np.random.default_rng(seed)
    for t in range(steps):
        n0 = [bk.n() for bk in p.oracle.books]
        forced = None
        if forced_every and t % forced_every == forced_every - 1:
            forced = [int(rng.integers(0, w.V + n0[b] + 1)) if p.oracle.books[b].prev is not None
                      else int(rng.integers(0, w.V)) for b in range(w.B)]
            # an id equal to V + n is legal only in the special case; keep forced ids existing
            forced = [min(z, w.V + n0[b] - 1) if n0[b] else min(z, w.V - 1)
                      for b, z in enumerate(forced)]
        if sits_out is not None:      # sequences that have finished take no part; the others run free
            forced = [zb.CODE_SELECTED] * w.B if forced is None else forced
            forced = [zb.CODE_NONE if sits_out(t, b) else z for b, z in enumerate(forced)]
        zb.z2z_decode_step(p.cb, g_hid[t], p.g_WE, p.g_WU, p.g_encE, p.g_encU, p.E_h, p.U_h,
                           select, 0.9, 4242, t,
                           None if forced is None else torch.tensor(forced, dtype=torch.int32,
                                                                    device=p.dev),
                           nxt, sel, lse, new, p.E_f32, p.U_f32, nxt_emb)
        if host_results:
            torch.cuda.synchronize()
        g_sel, g_nxt, g_lse, g_new = (x.cpu().numpy().copy() for x in (sel, nxt, lse, new))
        g_emb = f64(nxt_emb)
        sc = p.oracle.score(H[t], select, 0.9, 4242, t)
        apply = []
        for b in range(w.B):
            assert abs(g_lse[b] - sc[b]["lse"]) <= TOL, (t, b, g_lse[b], sc[b]["lse"])
            worst_lse = max(worst_lse, abs(g_lse[b] - sc[b]["lse"]))
            assert 0 <= g_sel[b] < w.V + n0[b]
            if g_sel[b] != sc[b]["choice"]:
                s = sc[b]["scores"]
                assert sc[b]["gap"] < GAP and s[g_sel[b]] >= s[sc[b]["choice"]] - GAP, \
                    (t, b, g_sel[b], sc[b]["choice"], sc[b]["gap"])
                followed += 1
            want_next = forced[b] if forced is not None and forced[b] != zb.CODE_SELECTED else int(g_sel[b])
            assert g_nxt[b] == want_next
            apply.append(want_next)
        onew = p.oracle.advance(apply, active=[z != zb.CODE_NONE for z in apply])
        assert g_new.tolist() == onew, (t, g_new.tolist(), onew)
        # input embedding of the applied codes for the next model step (Figure 2a): a base token's
        # row is a copy; a hypertoken's row is the cached hyper-embedding (the row created by this
        # very step included), held to the tolerance of the hyper-encoder
        E_pad = np.zeros((w.B, max(w.cap, 1), w.d))
        for b in range(w.B):
            E_pad[b, :p.oracle.E_h[b].shape[0]] = p.oracle.E_h[b]
        want_emb, bad = oemb.lookup(apply, None, f64(p.W_E), E_pad, [bk.n() for bk in p.oracle.books])
        assert bad == []
        for b in range(w.B):
            if apply[b] < w.V:                   # (a sequence that sat out: a zero row)
                assert np.array_equal(g_emb[b], want_emb[b])
            else:
                assert np.abs(g_emb[b] - want_emb[b]).max() <= TOL, (t, b, apply[b])
        for b in range(w.B):
            if onew[b] >= 0:
                p.check_cache_rows(b, onew[b], onew[b] + 1)
                p.force_caches_from_oracle(b, onew[b], onew[b] + 1)
        st, n = zb.z2z_status(p.cb)
        assert n.tolist() == [bk.n() for bk in p.oracle.books]
    p.check_codebooks()
    st, _ = zb.z2z_status(p.cb)
    assert all(int(x) & zb.ST_BAD_TOKEN == 0 for x in st)       # no step fed a code that names nothing
    return followed, worst_lse


def test_decode_step_tiny_config_argmax():
    followed, worst = _decode_follow(si.WORKLOADS["tiny"], 21, zb.SELECT_ARGMAX)
    print(f"tiny: followed {followed} near-ties, worst |LSE error| {worst:.2e}")


@pytest.mark.parametrize("w", [si.WORKLOADS["tiny"].scaled(name="tiny_b130", B=130, T=48, cap=24, steps=3),
                               SMALL_BF16.scaled(name="small_b130", B=130, T=40, cap=16, d=128, enc_dff=256, enc_heads=1,
                                                 steps=2)], ids=lambda w: w.name)
def test_decode_step_with_more_than_128_sequences(w):
    # beyond 128 sequences the step takes separate launches for merge, selection, LZW update and the
    # encoder's work list instead of the single fused update kernel
    _decode_follow(w, 47, zb.SELECT_ARGMAX, steps=w.steps)
    _decode_follow(w, 48, zb.SELECT_GUMBEL, steps=2, forced_every=2)


def test_decode_step_with_frozen_codebooks():
    # cap reached during the prompt: no step creates an entry, the hyper-encoder GEMMs find no live
    # entry and leave early; selections, LSE and the (unchanged) caches must still match
    w = SMALL_BF16.scaled(name="frozen", cap=24)
    p = Pair(w, seed=41)
    _prefill_both(p)
    assert all(bk.n() == w.cap for bk in p.oracle.books)
    _decode_follow(w, 41, zb.SELECT_ARGMAX, steps=5)
    _decode_follow(w, 42, zb.SELECT_GUMBEL, steps=4, forced_every=2)
    # ... and once the host has seen that everything is full the encoder pass is not launched at all
    hid = si.make_hidden(w, 4 * w.B, 43).view(4, w.B, w.d).to(p.dev)
    nxt = torch.zeros(w.B, dtype=torch.int32, device=p.dev)
    per_step = []
    for t in range(4):
        zb.z2z_profile_read(p.cb)
        zb.z2z_decode_step(p.cb, hid[t], p.g_WE, p.g_WU, p.g_encE, p.g_encU, p.E_h, p.U_h, zb.SELECT_ARGMAX, 1.0,
                           0, t, None, nxt, None, None)
        _, launches = zb.z2z_profile_read(p.cb)              # waits for the stream
        per_step.append(launches)
    assert per_step[0]["encoder_gemm"] > 0                    # the step that reports the state still runs the pass
    assert all(s["encoder_gemm"] == 0 and s["encoder_other"] == 0 for s in per_step[1:]), per_step
    # a new session on the same handle starts unfrozen
    zb.z2z_codebook_init(p.cb)
    zb.z2z_profile_read(p.cb)
    zb.z2z_decode_step(p.cb, hid[0], p.g_WE, p.g_WU, p.g_encE, p.g_encU, p.E_h, p.U_h, zb.SELECT_ARGMAX, 1.0,
                       0, 0, None, nxt, None, None)
    _, launches = zb.z2z_profile_read(p.cb)
    assert launches["encoder_gemm"] > 0


def test_decode_step_codebooks_fill_up_during_decode():
    # The cap is reached in the middle of decoding.  The step that creates a sequence's last entry
    # must still embed it on both sides (its rows are held against the oracle inside _decode_follow),
    # and the hyper-encoder pass runs in every step that can still create an entry, never afterwards:
    # the host samples the "all full" word before it enqueues a step, and a step only reports
    # codebooks that were already full when it began.
    base = SMALL_BF16
    seed = 44
    tokens = si.make_tokens(base, seed)
    n_prompt = [olzw.encode(tokens[b].tolist(), base.V, base.M, 10 ** 6)[2].n() for b in range(base.B)]
    w = base.scaled(name="fills_up", cap=min(n_prompt) + 2)
    _decode_follow(w, seed, zb.SELECT_ARGMAX, steps=10)            # checks every created row, the last one included
    p = Pair(w, seed=seed)
    _prefill_both(p)
    assert min(bk.n() for bk in p.oracle.books) == w.cap - 2
    hid = si.make_hidden(w, 16 * w.B, seed + 1).view(16, w.B, w.d).to(p.dev)
    nxt = torch.zeros(w.B, dtype=torch.int32, device=p.dev)
    new = torch.zeros(w.B, dtype=torch.int32, device=p.dev)
    passes, full_before = [], []
    for t in range(16):
        _, n = zb.z2z_status(p.cb)
        full_before.append(bool((n >= w.cap).all()))
        zb.z2z_profile_read(p.cb)
        zb.z2z_decode_step(p.cb, hid[t], p.g_WE, p.g_WU, p.g_encE, p.g_encU, p.E_h, p.U_h, zb.SELECT_ARGMAX, 1.0,
                           0, t, None, nxt, None, None, new, p.E_f32, p.U_f32)
        _, launches = zb.z2z_profile_read(p.cb)                 # waits for the stream
        passes.append(launches["encoder_gemm"] > 0)
        for b in range(w.B):                                    # a created row was written on both sides
            k = int(new[b].item())
            if k >= 0:
                assert float(p.E_f32[b, k].abs().max().item()) > 0 and float(p.U_f32[b, k].abs().max().item()) > 0
    assert full_before[-1] and not full_before[0]               # the codebooks filled up on the way
    first_full = full_before.index(True)
    # not full before the step -> the pass ran; the first step that starts full reports it (and may
    # still run the pass); every later step launches none
    assert all(passes[:first_full]), (passes, full_before)
    assert not any(passes[first_full + 1:]), (passes, full_before)


def test_decode_step_results_written_to_pinned_host_memory():
    for w, sel in ((si.WORKLOADS["tiny"], zb.SELECT_ARGMAX), (SMALL_BF16, zb.SELECT_GUMBEL)):
        _decode_follow(w, 27, sel, steps=6, forced_every=3, host_results=True)


@pytest.mark.parametrize("w", [SMALL_BF16.scaled(name="small_bf16_b5", B=5),
                               si.WORKLOADS["tiny"].scaled(name="tiny_b130", B=130, T=48, cap=24)],
                         ids=lambda w: w.name)
def test_decode_step_with_sequences_sitting_out(w):
    # a batch whose sequences finish at different times: a finished sequence keeps its codebook,
    # caches and status while the others go on (free-running and teacher-forced steps mixed);
    # 130 sequences take the path with separate selection and update kernels
    done_at = {b: 2 + (b % 4) for b in range(w.B)}
    _decode_follow(w, 61, zb.SELECT_ARGMAX, steps=7, forced_every=3,
                   sits_out=lambda t, b: b % 2 == 1 and t >= done_at[b])
    _decode_follow(w, 62, zb.SELECT_GUMBEL, steps=5, sits_out=lambda t, b: t % 2 == 1 and b != 0)


def test_decode_steps_replayed_from_a_cuda_graph():
    # the step only enqueues work on the caller's stream, so a caller may capture it: six steps
    # captured once and replayed give the session that six plain calls give (plain calls are the
    # ones held against the oracle above); floating-point results agree to summation order
    w, steps = SMALL_BF16, 6
    hid = si.make_hidden(w, (steps + 1) * w.B, 78).view(steps + 1, w.B, w.d).to(DEV)
    out = []
    for mode in ("plain", "graph"):
        p = Pair(w, seed=77)
        p.gpu_encode()
        total = w.B * w.cap
        zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, total, p.E_h, None)
        zb.z2z_hyper_embed(p.cb, zb.CACHE_UNEMBED, p.g_WU, p.g_encU, None, None, total, p.U_h, None)
        nxt = torch.zeros(steps + 1, w.B, dtype=torch.int32, device=DEV)
        new = torch.zeros(steps + 1, w.B, dtype=torch.int32, device=DEV)
        lse = torch.zeros(steps + 1, w.B, dtype=torch.float32, device=DEV)

        def step(t):
            zb.z2z_decode_step(p.cb, hid[t], p.g_WE, p.g_WU, p.g_encE, p.g_encU, p.E_h, p.U_h,
                               zb.SELECT_GUMBEL, 0.9, 4242, t, None, nxt[t], None, lse[t], new[t])
        step(0)                                  # every kernel has run once before the capture
        torch.cuda.synchronize()
        if mode == "plain":
            for t in range(1, steps + 1):
                step(t)
        else:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for t in range(1, steps + 1):
                    step(t)
            torch.cuda.synchronize()
            assert int(nxt[1:].abs().sum().item()) == 0          # capturing ran nothing
            g.replay()
        torch.cuda.synchronize()
        st, n = zb.z2z_status(p.cb)
        books = [p.gpu_codebook(b)[0] for b in range(w.B)]
        out.append((nxt.cpu(), new.cpu(), lse.cpu(), n.tolist(), st.tolist(), books, p.E_h.float().cpu(),
                    p.U_h.float().cpu()))
    a, b = out
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert a[3] == b[3] and a[4] == b[4] == [0] * w.B and a[5] == b[5]
    assert int((a[1][1:] >= 0).sum()) > 0                        # the replayed steps created entries
    assert float((a[2] - b[2]).abs().max()) <= 1e-3
    for x, y in ((a[6], b[6]), (a[7], b[7])):
        assert float((x - y).abs().max()) <= 2.0 ** -6 * max(1.0, float(x.abs().max()))


def test_decode_step_tiny_config_sampling_and_forcing():
    _decode_follow(si.WORKLOADS["tiny"], 22, zb.SELECT_GUMBEL, forced_every=3)


@pytest.mark.parametrize("w", [SMALL_BF16, SMALL_FP32, SMALL_BF16.scaled(name="tied", tied=1),
                               SMALL_BF16.scaled(name="attn_only", enc_layers=1, enc_ffn=0),
                               SMALL_BF16.scaled(name="attn_only_2", enc_layers=2, enc_ffn=0)],
                         ids=lambda w: w.name)
def test_decode_step_small(w):
    _decode_follow(w, 23, zb.SELECT_ARGMAX, steps=w.steps)
    _decode_follow(w, 24, zb.SELECT_GUMBEL, steps=6, forced_every=2)


# ------------------------------------------------------------------------------------------------
# Second on-GPU path: the CUDA-core kernels on a bf16 session (tensor cores switched off), and
# shapes that exercise more than one 128-row tile of the tensor-core kernels
# ------------------------------------------------------------------------------------------------
def test_cuda_core_kernels_on_bf16_session():
    p = Pair(SMALL_BF16, seed=5, tensor_cores=False)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    _logits_case(SMALL_BF16, 11, [70, 0, 5], True, 1, tensor_cores=False)
    _decode_follow(SMALL_BF16, 23, zb.SELECT_ARGMAX, steps=6, tensor_cores=False)


MID_BF16 = si.Workload("mid_bf16", V=5000, d=384, dtype="bf16", B=40, T=96, M=3, cap=64,
                       zipf_s=1.1, copy_p=0.4, seg_min=3, seg_max=10, steps=4, enc_layers=2,
                       enc_heads=3, enc_dff=768)


def test_tensor_core_kernels_many_rows_and_sequences():
    # 40 sequences: decode rows 120 (> 64: hi and lo run as two MMAs), prefill passes span many
    # 128-row tiles, logits with several hundred hidden rows span several row tiles
    p = Pair(MID_BF16, seed=31)
    _, worst = _prefill_both(p)
    print(f"mid_bf16: max |hyper-embedding error| = {worst:.3e}")
    worst = _logits_case(MID_BF16, 32, [9] * MID_BF16.B, True, 1)
    print(f"mid_bf16: max |logit error| = {worst:.3e}")
    _decode_follow(MID_BF16, 33, zb.SELECT_ARGMAX, steps=4)


@pytest.mark.parametrize("w", [MID_BF16.scaled(name="wide_b40", d=512, enc_dff=1024, enc_heads=4, steps=3),
                               MID_BF16.scaled(name="wide_b24", B=24, d=256, enc_dff=512, enc_heads=2, steps=3)],
                         ids=lambda w: w.name)
def test_weight_streaming_gemm_with_many_rows_in_one_box(w):
    # decode passes of 120 / 72 rows: hi and lo rows side by side are more than 128 columns of one
    # MMA (N = 240 / 144), one k-block per stage
    assert 2 * w.B * w.M > 128
    _decode_follow(w, 37, zb.SELECT_ARGMAX, steps=w.steps)
    _decode_follow(w, 38, zb.SELECT_GUMBEL, steps=2)      # 24 rows: sampled on the decode-batch logits kernel


ROWS_BF16 = si.Workload("rows_bf16", V=3000, d=256, dtype="bf16", B=2, T=220, M=3, cap=80,
                        zipf_s=1.1, copy_p=0.4, seg_min=3, seg_max=10, steps=3, enc_layers=2,
                        enc_heads=2, enc_dff=512)


@pytest.mark.parametrize("w", [ROWS_BF16, ROWS_BF16.scaled(name="rows_bf16_m5", M=5, cap=45, B=3)],
                         ids=lambda w: w.name)
def test_weight_streaming_gemm_with_several_row_tiles(w):
    # passes of 480 / 675 rows: below the size of the CTA-pair GEMM and above one 128-row tile, so
    # the packed rows span several row tiles (one 256-row operand box each) and the last is ragged
    assert 128 < w.B * w.cap * w.M < 1024
    p = Pair(w, seed=35)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    print(f"{w.name}: max |hyper-embedding error| = {worst:.3e}")
    _decode_follow(w, 36, zb.SELECT_ARGMAX, steps=3)


@pytest.mark.parametrize("w", [SMALL_BF16.scaled(name="pair_m5", M=5, B=2, cap=240, T=900),
                               SMALL_BF16.scaled(name="pair_dh256", d=512, enc_heads=2, enc_dff=1024, B=3, cap=120, T=420)],
                         ids=lambda w: w.name)
def test_prompt_sized_pass_with_long_entries_and_wide_heads(w):
    # passes of >= 1024 rows (CTA-pair GEMMs, packed rows) whose attention does not fit the
    # registers of one warp: merge size 5, or heads of 256 columns
    assert w.B * w.cap * w.M >= 1024
    p = Pair(w, seed=45)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    print(f"{w.name}: max |hyper-embedding error| = {worst:.3e}")


def _embed_all_both_sides(p, max_entries):
    w = p.w
    p.E_f32.zero_(); p.U_f32.zero_()
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, max_entries, p.E_h, p.E_f32)
    zb.z2z_hyper_embed(p.cb, zb.CACHE_UNEMBED, p.g_WU, p.g_encU, None, None, max_entries, p.U_h, p.U_f32)
    worst = max(p.check_cache_rows(b, 0, p.oracle.books[b].n()) for b in range(w.B))
    return worst, p.E_f32.clone(), p.U_f32.clone()


@pytest.mark.parametrize("w", [SMALL_BF16.scaled(name="half_m4", B=5, cap=1000, T=1300),
                               SMALL_BF16.scaled(name="half_m5_dh256", M=5, d=512, enc_heads=2, enc_dff=1024, B=5,
                                                 cap=1000, T=1000),
                               SMALL_BF16.scaled(name="half_attn_only", enc_layers=2, enc_ffn=0, B=5, cap=1000, T=1100)],
                         ids=lambda w: w.name)
def test_prompt_sized_passes_with_a_single_fp16_operand(w):
    # z2z_set_encoder_half_scratch: calls that span several prompt-sized passes copy the encoder's
    # linear-layer weights to fp16 and round each activation once to fp16 (one MMA per k-step).  Held
    # to the same tolerance as the two-part form, against the same oracle rows.
    p = Pair(w, seed=48)
    codes, clen, after = p.gpu_encode()
    ocodes, _ = p.oracle.prefill([p.tokens[b].tolist() for b in range(w.B)])
    for b in range(w.B):
        assert codes[b, :clen[b]].tolist() == ocodes[b]
    bound = w.B * w.cap                                        # 5 passes of 1024 entries each
    worst2, E2, U2 = _embed_all_both_sides(p, bound)
    zb.z2z_profile_read(p.cb)
    scratch = torch.empty(zb.encoder_half_bytes(p.cfg) + 256, dtype=torch.uint8, device=DEV)
    scratch = scratch[(-scratch.data_ptr()) % 256:][:zb.encoder_half_bytes(p.cfg)]
    zb.z2z_set_encoder_half_scratch(p.cb, scratch)
    zb.z2z_codebook_init(p.cb)                                 # same handle, new session: embed everything again
    p.gpu_encode()
    p.E_h.zero_(); p.U_h.zero_()
    worst1, E1, U1 = _embed_all_both_sides(p, bound)
    assert worst1 <= TOL and worst2 <= TOL
    assert not torch.equal(E1, E2) and not torch.equal(U1, U2)            # the other arithmetic really ran
    assert worst1 >= worst2                                     # 11 mantissa bits against about 16
    print(f"{w.name}: max |hyper-embedding error| two-part {worst2:.3e}, single fp16 operand {worst1:.3e}")
    st, _ = zb.z2z_status(p.cb)
    assert int(st.max()) & zb.ST_HALF_RANGE == 0
    # short calls (fewer than four passes) keep the two-part form: bit-identical to the first run
    zb.z2z_codebook_init(p.cb)
    p.gpu_encode()
    assert sum(bk.n() for bk in p.oracle.books) <= 3 * 1024
    worst3, E3, U3 = _embed_all_both_sides(p, 3 * 1024)
    assert torch.equal(E3, E2) and torch.equal(U3, U2)
    # ... and without the scratch everything is as before
    zb.z2z_set_encoder_half_scratch(p.cb, None)
    zb.z2z_codebook_init(p.cb)
    p.gpu_encode()
    worst4, E4, U4 = _embed_all_both_sides(p, bound)
    assert worst4 == worst2


def test_half_scratch_reports_weights_beyond_fp16_range():
    w = SMALL_BF16.scaled(name="half_range", B=5, cap=1000, T=600)
    p = Pair(w, seed=49)
    p.gpu_encode()
    scratch = torch.empty(zb.encoder_half_bytes(p.cfg) + 256, dtype=torch.uint8, device=DEV)
    scratch = scratch[(-scratch.data_ptr()) % 256:][:zb.encoder_half_bytes(p.cfg)]
    zb.z2z_set_encoder_half_scratch(p.cb, scratch)
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, w.B * w.cap, p.E_h, None)
    st, _ = zb.z2z_status(p.cb)
    assert int(st.max()) & zb.ST_HALF_RANGE == 0
    p.g_encE_t[1 + 8][3, 5] = 1.0e6                             # W1 of layer 0: not representable in fp16
    zb.z2z_hyper_embed(p.cb, zb.CACHE_EMBED, p.g_WE, p.g_encE, None, None, w.B * w.cap, p.E_h, None)
    st, _ = zb.z2z_status(p.cb)
    assert all(int(x) & zb.ST_HALF_RANGE for x in st)
    with pytest.raises(zb.Z2ZError, match="aligned"):
        zb.z2z_set_encoder_half_scratch(p.cb, scratch[8:])


def test_attention_only_layers_on_every_encoder_path():
    # layers without a feed-forward block (enc_dff = 0): the CUDA-core kernels on a bf16 session,
    # the weight-streaming GEMM with several row tiles, and a prompt-sized pass (CTA-pair GEMMs)
    w = SMALL_BF16.scaled(name="attn_only_2", enc_layers=2, enc_ffn=0)
    assert w.dff == 0
    p = Pair(w, seed=5, tensor_cores=False)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    w = ROWS_BF16.scaled(name="rows_attn_only", enc_ffn=0)
    p = Pair(w, seed=35)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    w = SMALL_BF16.scaled(name="pair_attn_only", enc_layers=2, enc_ffn=0, B=2, cap=300, T=1100)
    assert w.B * w.cap * w.M >= 1024
    p = Pair(w, seed=46)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    print(f"{w.name}: max |hyper-embedding error| = {worst:.3e}")


# ------------------------------------------------------------------------------------------------
# Prompt-scoring logits kernel (CTA pairs, 256 x 256 tiles), forced on for small shapes:
# several row tiles with a ragged tail, rows of several sequences inside one tile, sequences
# without rows, causal per-row limits, every number of column strips, both epilogue paths
# ------------------------------------------------------------------------------------------------
PAIR_BF16 = si.Workload("pair_bf16", V=3000, d=256, dtype="bf16", B=5, T=1400, M=3, cap=700,
                        zipf_s=1.1, copy_p=0.5, seg_min=3, seg_max=10, steps=0, enc_layers=0,
                        enc_heads=2, enc_dff=512)


@pytest.mark.parametrize("strips", [0, 1, 3, 8])
def test_pair_logits_kernel_fast_path(strips):
    # reductions only: the epilogue that folds whole 256-column tiles; hypertokens need > 1 tile
    rows = [300, 0, 77, 256, 130]
    worst = _logits_case(PAIR_BF16, 41, rows, False, 0, tensor_cores=2 + 16 * strips, debug=False)
    print(f"pair kernel, strips={strips}: max |LSE error| = {worst:.3e}")


@pytest.mark.parametrize("strips,causal,select", [(0, True, 1), (2, False, 1), (8, True, 0)])
def test_pair_logits_kernel_generic_path(strips, causal, select):
    rows = [40, 0, 300, 5, 200]
    worst = _logits_case(PAIR_BF16, 42, rows, causal, select, tensor_cores=2 + 16 * strips)
    print(f"pair kernel (all outputs), strips={strips}: max |logit error| = {worst:.3e}")


def test_pair_logits_kernel_causal_fast_path_and_no_hypertokens():
    _logits_case(PAIR_BF16, 43, [256, 256, 1, 0, 90], True, 0, tensor_cores=2, debug=False)
    _logits_case(PAIR_BF16.scaled(cap=0, name="pair_nocap"), 44, [100, 200, 0, 0, 3], False, 0,
                 tensor_cores=2, debug=False)


# ------------------------------------------------------------------------------------------------
# Decode logits kernel (weight rows as the MMA's M operand, one thread per vocabulary row, fixed
# shares plus a claimed pool): every batch-size class, hidden rows resident in shared memory or
# streamed per stage, rows that share a sequence, causal limits, all outputs, repeated launches
# (the pool counter must come back to zero)
# ------------------------------------------------------------------------------------------------
WIDE_BF16 = si.Workload("wide_bf16", V=2000, d=1280, dtype="bf16", B=4, T=600, M=3, cap=300,
                        zipf_s=1.1, copy_p=0.5, seg_min=3, seg_max=10, steps=0, enc_layers=0,
                        enc_heads=2, enc_dff=512)
TALL_BF16 = si.Workload("tall_bf16", V=40000, d=256, dtype="bf16", B=6, T=900, M=3, cap=500,
                        zipf_s=1.1, copy_p=0.5, seg_min=3, seg_max=10, steps=0, enc_layers=0,
                        enc_heads=2, enc_dff=512)


@pytest.mark.parametrize("rows,causal,select,debug", [
    ([2, 1, 3, 1, 1], False, 0, False),      # 8 rows, reductions only
    ([3, 0, 5, 4, 1], True, 1, True),        # 13 rows -> 16-row class, sampling + all outputs
    ([16, 0, 0, 0, 0], True, 0, True),       # one sequence owns every row
    ([7, 7, 5, 5, 5], False, 0, False),      # 29 rows -> 32-row class
    ([6, 6, 6, 7, 7], True, 0, False),       # 32 rows, causal
    ([7, 7, 5, 5, 5], True, 1, True),        # 29 rows: sampling and every output, two warps per lane quarter
    ([6, 6, 6, 7, 7], False, 1, True),       # 32 rows, sampling and every output
    ([0, 17, 0, 0, 0], True, 1, False),      # 17 rows of one sequence, sampling without the debug outputs
])
def test_decode_logits_kernel_batches(rows, causal, select, debug):
    worst = _logits_case(PAIR_BF16, 51, rows, causal, select, debug=debug)
    print(f"decode kernel rows={sum(rows)}: worst error {worst:.3e}")


@pytest.mark.parametrize("rows,select,debug", [([8, 8, 8, 8], 0, False), ([2, 6, 3, 5], 1, True)])
def test_decode_logits_kernel_streamed_hidden_rows(rows, select, debug):
    # d = 1280: 32 (16) rows x 20 k-blocks exceed (fit) the resident budget
    _logits_case(WIDE_BF16, 52, rows, True, select, debug=debug)


def test_decode_logits_kernel_fixed_shares_and_pool():
    # V = 40000: every CTA owns a fixed share of 128-row jobs and the pool holds both W_U and U_h
    _logits_case(TALL_BF16, 53, [1, 1, 1, 1, 1, 1], False, 0, debug=False)
    _logits_case(TALL_BF16, 54, [2, 3, 1, 4, 0, 2], True, 1, debug=True)
    _logits_case(TALL_BF16, 55, [5, 6, 4, 7, 3, 6], True, 1, debug=True)        # 31 rows, sampled


# ------------------------------------------------------------------------------------------------
# Limits of the configuration: largest and smallest merge size through the encoder and the decode
# step, the largest batch, the largest codebook
# ------------------------------------------------------------------------------------------------
def _periodic_tail(p: Pair, period: int, head: int):
    """Everything after the first `head` tokens of a prompt becomes a short cycle, so that phrases
    reach length M."""
    w = p.w
    t = p.tokens.copy()
    for b in range(w.B):
        t[b, head:] = (np.arange(w.T - head) % period) + 3 * b
    p.tokens = t


@pytest.mark.parametrize("w", [SMALL_BF16.scaled(name="m8_bf16", M=8, T=400, cap=200, B=2, steps=4),
                               SMALL_FP32.scaled(name="m8_fp32", M=8, T=300, cap=120, B=2, steps=3),
                               SMALL_BF16.scaled(name="m8_small_pass", M=8, T=120, cap=63, B=2, steps=2),
                               SMALL_BF16.scaled(name="m2_bf16", M=2, steps=3)],
                         ids=lambda w: w.name)
def test_hyper_embed_at_the_merge_size_limits(w):
    p = Pair(w, seed=51)
    if w.name == "m8_small_pass":              # < 1024 rows per pass: the weight-streaming GEMM
        assert w.B * w.cap * w.M < 1024
        _periodic_tail(p, 2, 30)
    else:
        _periodic_tail(p, 5, w.T // 2)
    _, worst = _prefill_both(p)
    assert worst <= TOL
    longest = max(len(e) for bk in p.oracle.books for e in bk.entries)
    assert longest == w.M
    print(f"{w.name}: max |hyper-embedding error| = {worst:.3e}, longest entry {longest}")


@pytest.mark.parametrize("w", [SMALL_BF16.scaled(name="m8_bf16", M=8, T=400, cap=200, B=2, copy_p=0.7,
                                                 seg_min=8, seg_max=40),
                               SMALL_BF16.scaled(name="m1_bf16", M=1),
                               SMALL_FP32.scaled(name="m1_fp32", M=1)],
                         ids=lambda w: w.name)
def test_decode_step_at_the_merge_size_limits(w):
    # M = 1 never creates a hypertoken: the step is a plain LM-head selection and the codebooks
    # stay empty; M = 8 is the largest merge size
    _decode_follow(w, 53, zb.SELECT_ARGMAX, steps=4)
    if w.M == 1:
        p = Pair(w, seed=53)
        p.gpu_encode()
        assert zb.z2z_status(p.cb)[1].tolist() == [0] * w.B


@pytest.mark.parametrize("w", [si.WORKLOADS["tiny"].scaled(name="tiny_b1024", B=1024, T=24, cap=8, steps=2),
                               SMALL_BF16.scaled(name="bf16_b1024", B=1024, T=24, cap=8, d=128, enc_heads=1,
                                                 enc_dff=256, steps=2)],
                         ids=lambda w: w.name)
def test_largest_batch(w):
    _decode_follow(w, 55, zb.SELECT_ARGMAX, steps=w.steps)


def test_largest_codebook():
    # cap = 65535, the most the 16-bit entry field of a slot addresses: nearly every pair of a
    # uniform stream over a large vocabulary is new, so the book fills and freezes
    rng = np.random.default_rng(57)
    tokens = rng.integers(0, 60000, size=(1, 80000)).astype(np.int32)
    g = _compare_encode(60000, 3, 65535, tokens)
    ents, st = g.entries(0)
    assert len(ents) == 65535 and st & zb.ST_CAP_FROZEN

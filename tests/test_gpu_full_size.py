"""Parity at the FULL sizes of the benchmark configurations, in the launch configuration the
benchmark times (z2z_decode_step for the decode workloads; encode + hyper-embed + joint logits over
every compressed position for the prompt-scoring workload).  At these sizes the fp64 oracle cannot
produce every output, so it computes sampled ones, one by one:

  * the joint-logit reductions (LSE, argmax with the top-2 gap rule) of sampled hidden rows, the
    static part taken block by block through the oracle's own joint_logits;
  * the hyper-embedding of sampled new codebook entries (oracle LZW replayed for that sequence,
    oracle hyper-encoder on the gathered rows).

No oracle input comes from the CUDA path: the hyper-unembedding cache that the logits read is
filled with generator values on both sides, the codebooks come from the oracle's own LZW.
"""
import numpy as np
import pytest
import torch

from oracle import hyper_encoder as ohe, logits as olg, lzw as olzw
from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import synth_inputs as si
from tests._harness import GAP, TOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


def _oracle_logits(h64, W_U, U_rows64, block=16384):
    """Joint logits of one hidden row; W_U (bf16/fp32 torch, CPU) is converted block by block."""
    parts = [olg.joint_logits(h64, _f64(W_U[i:i + block]), None) for i in range(0, W_U.shape[0], block)]
    l = np.concatenate(parts)
    if U_rows64 is not None and U_rows64.shape[0] > 0:
        l = np.concatenate([l, U_rows64 @ h64])
    return l


def _oracle_embed(entry, table, enc64, heads):
    """Oracle hyper-encoder on one entry; only the gathered rows of the table are converted."""
    ids = [int(t) for t in entry]
    small = _f64(table[ids])
    return ohe.hyper_embed_one(list(range(len(ids))), small, enc64, heads)


class FullSession:
    def __init__(self, w, seed):
        self.w = w
        self.tokens = si.make_tokens(w, seed)
        self.W_E, self.W_U = si.make_tables(w, seed)
        self.enc_E = si.make_encoder(w, seed * 3 + 1)
        self.enc_U = si.make_encoder(w, seed * 3 + 2)
        self.cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, w.enc_layers, w.heads, w.dff, 0)
        self.cb = zb.Codebook(self.cfg, DEV)
        self.g_WE, self.g_WU = self.W_E.to(DEV), self.W_U.to(DEV)
        self.g_encE_t = [t.to(DEV) for t in self.enc_E]
        self.g_encU_t = [t.to(DEV) for t in self.enc_U]
        self.g_encE, self.g_encU = zb.encoder_weights(self.g_encE_t), zb.encoder_weights(self.g_encU_t)
        # hyper-unembedding rows straight from the generator: identical values on both sides
        # (at most 8 distinct blocks, repeated over the sequences, to bound the host's generation time)
        base = si.normal_tensor((min(w.B, 8), w.cap, w.d), 0.05, seed + 100, w.torch_dtype)
        self.U_syn = base[torch.arange(w.B) % base.shape[0]]
        self.U_h = self.U_syn.to(DEV)
        self.E_h = torch.zeros(w.B, w.cap, w.d, dtype=w.torch_dtype, device=DEV)
        g_tok = torch.from_numpy(self.tokens).to(DEV)
        self.codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=DEV)
        self.clen = torch.zeros(w.B, dtype=torch.int32, device=DEV)
        self.after = torch.zeros(w.B, w.T, dtype=torch.int32, device=DEV)
        zb.z2z_lzw_encode(self.cb, g_tok, None, self.codes, self.clen, self.after)
        self.books = {}

    def book(self, b):
        """Oracle codebook of sequence b after its prompt (computed on demand)."""
        if b not in self.books:
            w = self.w
            _, _, ob = olzw.encode(self.tokens[b].tolist(), w.V, w.M, w.cap)
            self.books[b] = ob
        return self.books[b]


@pytest.mark.parametrize("name,steps,sample_seqs", [("phi3_mini_head", 3, [0, 5, 7]),
                                                    ("llama3_8b_head", 2, [0, 17, 31]),
                                                    ("long_context", 2, [1, 3])])
def test_full_size_decode_steps_sampled(name, steps, sample_seqs):
    w = si.WORKLOADS[name]
    s = FullSession(w, seed=71)
    st, n_gpu = zb.z2z_status(s.cb)
    for b in sample_seqs:
        assert int(n_gpu[b]) == s.book(b).n()
    hid = si.make_hidden(w, steps * w.B, 72).view(steps, w.B, w.d)
    g_hid = hid.to(DEV)
    nxt = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    sel = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    lse = torch.zeros(w.B, dtype=torch.float32, device=DEV)
    new = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    E32 = torch.zeros(w.B, w.cap, w.d, dtype=torch.float32, device=DEV)
    U32 = torch.zeros_like(E32)
    encE64 = [_f64(t) for t in s.enc_E]
    encU64 = [_f64(t) for t in s.enc_U]
    U_seen = {b: _f64(s.U_syn[b]) for b in sample_seqs}        # rows the logits of sequence b read
    worst_lse = worst_emb = 0.0
    for t in range(steps):
        zb.z2z_decode_step(s.cb, g_hid[t], s.g_WE, s.g_WU, s.g_encE, s.g_encU, s.E_h, s.U_h,
                           zb.SELECT_ARGMAX, 1.0, 0, t, None, nxt, sel, lse, new, E32, U32)
        g_sel, g_lse, g_new = sel.cpu().numpy(), lse.cpu().numpy(), new.cpu().numpy()
        for b in sample_seqs:
            ob = s.book(b)
            nb = ob.n()
            l = _oracle_logits(_f64(hid[t, b]), s.W_U, U_seen[b][:nb])
            want = olg.lse(l)
            worst_lse = max(worst_lse, abs(g_lse[b] - want))
            assert abs(g_lse[b] - want) <= TOL, (name, t, b, g_lse[b], want)
            a, best, gap = olg.top2(l)
            assert 0 <= g_sel[b] < w.V + nb
            if g_sel[b] != a:
                assert gap < GAP and l[g_sel[b]] >= best - GAP, (name, t, b, g_sel[b], a, gap)
            k = ob.step(int(g_sel[b]))                           # oracle LZW update with the applied code
            assert g_new[b] == k, (name, t, b, g_new[b], k)
            if k >= 0:
                e_want = _oracle_embed(ob.entries[k], s.W_E, encE64, w.heads)
                u_want = _oracle_embed(ob.entries[k], s.W_U, encU64, w.heads)
                e_got = E32[b, k].cpu().double().numpy()
                u_got = U32[b, k].cpu().double().numpy()
                err = max(np.abs(e_got - e_want).max(), np.abs(u_got - u_want).max())
                worst_emb = max(worst_emb, err)
                assert err <= TOL, (name, t, b, err)
                assert torch.equal(s.E_h[b, k].cpu(), E32[b, k].cpu().to(w.torch_dtype))
                assert torch.equal(s.U_h[b, k].cpu(), U32[b, k].cpu().to(w.torch_dtype))
                # the next step's logits read the row the GPU stored; the oracle's own row, rounded
                # to the storage type, must agree with it within the tolerance just checked
                U_seen[b][k] = _f64(torch.from_numpy(u_want).to(w.torch_dtype))
                s.U_h[b, k] = torch.from_numpy(u_want).to(w.torch_dtype).to(DEV)
    st, _ = zb.z2z_status(s.cb)
    assert int(st.max()) & ~zb.ST_CAP_FROZEN == 0
    print(f"{name}: worst |LSE error| {worst_lse:.2e}, worst |hyper-embedding error| {worst_emb:.2e}")


def _oracle_logits_rows(H64, W_U, block=16384):
    """Static part of the joint logits of several hidden rows at once: the oracle's joint_logits
    applied to the rows as columns of one matrix, W_U converted to fp64 block by block.
    Returns [V, rows]."""
    parts = [olg.joint_logits(H64.T, _f64(W_U[i:i + block]), None) for i in range(0, W_U.shape[0], block)]
    return np.concatenate(parts, axis=0)


def test_full_size_prompt_scoring_sampled():
    """prefill_heavy at its full size (64 prompts of 8192 tokens): every compressed position scored
    against V + n_vis columns by the CTA-pair kernel with causal visibility from the encoder's
    entries_after.  The oracle scores a sample of positions chosen where an indexing mistake would
    show: the first and last row of 256-row tiles, rows on both sides of sequence boundaries that
    fall inside a tile, rows that see no hypertoken and rows that see all of them, plus random rows.
    Then both hyper-encoders run prompt-sized passes (all entries of two sequences, a few of every
    other) and a sample of entries, entries of length M among them, is held against the oracle."""
    w = si.WORKLOADS["prefill_heavy"]
    s = FullSession(w, seed=73)
    clen = s.clen.cpu().numpy()
    N = int(clen.sum())
    offs = np.concatenate([[0], np.cumsum(clen)]).astype(np.int64)
    row_seq = torch.repeat_interleave(torch.arange(w.B, dtype=torch.int32, device=DEV), s.clen.to(torch.int64))
    # visible hypertokens at compressed position i of sequence b: those that exist once code i is out
    mask = torch.arange(w.T, device=DEV)[None, :] < s.clen[:, None]
    row_nvis = s.after[mask].contiguous()
    assert row_seq.numel() == N and row_nvis.numel() == N
    st, n_gpu = zb.z2z_status(s.cb)
    rng = np.random.default_rng(75)
    n_tiles = (N + 255) // 256
    rows = set()
    for t in [0, 1, n_tiles // 3, n_tiles // 2, n_tiles - 2, n_tiles - 1]:
        rows.update([t * 256, min(t * 256 + 255, N - 1)])                 # tile edges (the last tile is ragged)
    inner = [b for b in range(1, w.B) if offs[b] % 256 not in (0, 255)]  # boundaries inside a tile
    for b in inner[:6] + inner[-2:]:
        rows.update([int(offs[b]) - 1, int(offs[b])])
    none_rows = [int(offs[b]) + int(rng.integers(1, clen[b])) for b in (2, 31, w.B - 1)]
    all_rows = [int(offs[b]) + int(rng.integers(0, clen[b] - 1)) for b in (0, 17, 40, w.B - 2)]
    rows.update(none_rows + all_rows)
    while len(rows) < 72:
        rows.add(int(rng.integers(0, N)))
    rows = sorted(rows)
    seq_of = np.searchsorted(offs, np.asarray(rows), side="right") - 1
    # two overrides of the causal limit (any value in [0, n_b] is a legal input): no hypertoken
    # visible, and every hypertoken of the sequence visible
    nvis_host = row_nvis.cpu().numpy().copy()
    for r in none_rows:
        nvis_host[r] = 0
    for r in all_rows:
        nvis_host[r] = s.book(int(np.searchsorted(offs, r, side="right") - 1)).n()
    row_nvis = torch.from_numpy(nvis_host).to(DEV)
    hid = si.make_hidden(w, 16384, 74)[torch.arange(N) % 16384]     # 16384 distinct rows, repeated
    g_hid = hid.to(DEV)
    lse = torch.zeros(N, dtype=torch.float32, device=DEV)
    am = torch.zeros(N, dtype=torch.int32, device=DEV)
    mx = torch.zeros(N, dtype=torch.float32, device=DEV)
    zb.z2z_dynamic_logits(s.cb, g_hid, row_seq, row_nvis, s.g_WU, s.U_h, zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                          lse, am, mx)
    g_lse, g_am, g_mx = lse.cpu().numpy(), am.cpu().numpy(), mx.cpu().numpy()
    H64 = _f64(hid[rows])
    static = _oracle_logits_rows(H64, s.W_U)                        # [V, len(rows)]
    enc_cache = {}
    worst = 0.0
    for x, r in enumerate(rows):
        b = int(seq_of[x]); i = r - int(offs[b])
        if b not in enc_cache:
            enc_cache[b] = olzw.encode(s.tokens[b].tolist(), w.V, w.M, w.cap)
        codes_b, after_b, ob = enc_cache[b]
        assert len(codes_b) == clen[b] and ob.n() == int(n_gpu[b])
        nv = 0 if r in none_rows else (ob.n() if r in all_rows else after_b[i])
        assert nv == nvis_host[r]
        l = static[:, x]
        if nv > 0:
            l = np.concatenate([l, _f64(s.U_syn[b, :nv]) @ H64[x]])
        want = olg.lse(l)
        worst = max(worst, abs(g_lse[r] - want))
        assert abs(g_lse[r] - want) <= TOL, (b, i, r, g_lse[r], want)
        a, best, gap = olg.top2(l)
        assert abs(g_mx[r] - best) <= TOL, (b, i, r)
        assert 0 <= g_am[r] < w.V + nv, (b, i, r, g_am[r], nv)
        if g_am[r] != a:
            assert gap < GAP and l[g_am[r]] >= best - GAP, (b, i, r)
    print(f"prefill_heavy: {N} rows scored, {len(rows)} sampled, worst sampled |LSE error| {worst:.2e}")
    del g_hid, lse, am, mx, static
    # ---- hyper-embedding at prompt size, both sides (CTA-pair GEMM passes)
    full = [5, 50]                                   # every entry of these sequences; four of every other
    nb = [s.book(b).n() if b in full else 0 for b in range(w.B)]
    first_h = [0 if b in full else int(rng.integers(0, 1000)) for b in range(w.B)]
    count_h = [nb[b] if b in full else 4 for b in range(w.B)]
    first = torch.tensor(first_h, dtype=torch.int32, device=DEV)
    count = torch.tensor(count_h, dtype=torch.int32, device=DEV)
    E32 = torch.zeros(w.B, w.cap, w.d, dtype=torch.float32, device=DEV)
    U_out = torch.zeros(w.B, w.cap, w.d, dtype=w.torch_dtype, device=DEV)
    zb.z2z_hyper_embed(s.cb, zb.CACHE_EMBED, s.g_WE, s.g_encE, first, count, sum(count_h), s.E_h, E32)
    picks = []
    for b in full:
        ents = s.book(b).entries
        longest = [k for k in range(len(ents)) if len(ents[k]) == w.M]
        assert longest
        ks = {0, len(ents) - 1, longest[0], longest[-1], longest[len(longest) // 2]}
        while len(ks) < 12:
            ks.add(int(rng.integers(0, len(ents))))
        picks += [(b, k) for k in sorted(ks)]
    picks += [(b, first_h[b] + j) for b, j in ((0, 0), (1, 3), (33, 2), (w.B - 1, 1), (20, 0), (41, 3), (63, 0), (12, 2))]
    assert len(picks) >= 32
    worst_e = 0.0
    for side, table, enc_t, cache, out32 in (("E", s.W_E, s.enc_E, s.E_h, E32), ("U", s.W_U, s.enc_U, U_out, None)):
        if side == "U":
            E32.zero_()                               # the one fp32 side buffer serves both sides in turn
            zb.z2z_hyper_embed(s.cb, zb.CACHE_UNEMBED, s.g_WU, s.g_encU, first, count, sum(count_h), U_out, E32)
        enc64 = [_f64(t) for t in enc_t]
        for b, k in picks:
            want = _oracle_embed(s.book(b).entries[k], table, enc64, w.heads)
            err = np.abs(E32[b, k].cpu().double().numpy() - want).max()
            worst_e = max(worst_e, err)
            assert err <= TOL, (side, b, k, err)
            assert torch.equal(cache[b, k].cpu(), E32[b, k].cpu().to(w.torch_dtype))
        if side == "E":
            # the same entries once more with a single fp16 operand per GEMM (weights copied to fp16,
            # activations rounded once): same oracle rows, same tolerance
            nbytes = zb.encoder_half_bytes(s.cfg)
            scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=DEV)
            scratch = scratch[(-scratch.data_ptr()) % 256:][:nbytes]
            zb.z2z_set_encoder_half_scratch(s.cb, scratch)
            E32.zero_()
            zb.z2z_hyper_embed(s.cb, zb.CACHE_EMBED, s.g_WE, s.g_encE, first, count, 8 * 1024, s.E_h, E32)
            worst_h = 0.0
            for b, k in picks:
                want = _oracle_embed(s.book(b).entries[k], table, enc64, w.heads)
                err = np.abs(E32[b, k].cpu().double().numpy() - want).max()
                worst_h = max(worst_h, err)
                assert err <= TOL, ("E, single fp16 operand", b, k, err)
                assert torch.equal(cache[b, k].cpu(), E32[b, k].cpu().to(w.torch_dtype))
            st, _ = zb.z2z_status(s.cb)
            assert int(st.max()) & zb.ST_HALF_RANGE == 0
            zb.z2z_set_encoder_half_scratch(s.cb, None)
            del scratch
            print(f"prefill_heavy: single fp16 operand, worst |hyper-embedding error| {worst_h:.2e}")
        del enc64
    print(f"prefill_heavy: {len(picks)} entries per side, worst |hyper-embedding error| {worst_e:.2e}")

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


def test_full_size_prompt_scoring_sampled():
    """prefill_heavy: every compressed position scored against V + n_b columns (CTA-pair kernel),
    causal visibility from the encoder's entries_after; a sample of entries embedded and checked."""
    w = si.WORKLOADS["prefill_heavy"]
    s = FullSession(w, seed=73)
    clen = s.clen.cpu().numpy()
    N = int(clen.sum())
    row_seq = torch.repeat_interleave(torch.arange(w.B, dtype=torch.int32, device=DEV), s.clen.to(torch.int64))
    # visible hypertokens at compressed position i of sequence b: those that exist once code i is out
    mask = torch.arange(w.T, device=DEV)[None, :] < s.clen[:, None]
    row_nvis = s.after[mask].contiguous()
    assert row_seq.numel() == N and row_nvis.numel() == N
    hid = si.make_hidden(w, 16384, 74)[torch.arange(N) % 16384]     # 16384 distinct rows, repeated
    g_hid = hid.to(DEV)
    lse = torch.zeros(N, dtype=torch.float32, device=DEV)
    am = torch.zeros(N, dtype=torch.int32, device=DEV)
    mx = torch.zeros(N, dtype=torch.float32, device=DEV)
    zb.z2z_dynamic_logits(s.cb, g_hid, row_seq, row_nvis, s.g_WU, s.U_h, zb.SELECT_ARGMAX, 1.0, 0, 0, None,
                          lse, am, mx)
    g_lse, g_am, g_mx = lse.cpu().numpy(), am.cpu().numpy(), mx.cpu().numpy()
    offs = np.concatenate([[0], np.cumsum(clen)])
    rng = np.random.default_rng(75)
    samples = [(0, 0), (0, int(clen[0]) - 1), (w.B - 1, int(clen[-1]) - 1)]
    samples += [(int(b), int(rng.integers(0, clen[b]))) for b in rng.integers(0, w.B, size=5)]
    worst = 0.0
    for b, i in samples:
        r = int(offs[b]) + i
        codes_b, after_b, _ = olzw.encode(s.tokens[b].tolist(), w.V, w.M, w.cap)
        assert len(codes_b) == clen[b]
        nv = after_b[i]
        l = _oracle_logits(_f64(hid[r]), s.W_U, _f64(s.U_syn[b, :nv]))
        worst = max(worst, abs(g_lse[r] - olg.lse(l)))
        assert abs(g_lse[r] - olg.lse(l)) <= TOL, (b, i, g_lse[r], olg.lse(l))
        a, best, gap = olg.top2(l)
        assert abs(g_mx[r] - best) <= TOL
        if g_am[r] != a:
            assert gap < GAP and l[g_am[r]] >= best - GAP
    print(f"prefill_heavy: {N} rows scored, worst sampled |LSE error| {worst:.2e}")
    # hyper-embedding of a sample of entries of every sequence (explicit ranges)
    first = torch.tensor([int(rng.integers(0, 1000)) for _ in range(w.B)], dtype=torch.int32, device=DEV)
    count = torch.full((w.B,), 4, dtype=torch.int32, device=DEV)
    E32 = torch.zeros(w.B, w.cap, w.d, dtype=torch.float32, device=DEV)
    zb.z2z_hyper_embed(s.cb, zb.CACHE_EMBED, s.g_WE, s.g_encE, first, count, 4 * w.B, s.E_h, E32)
    encE64 = [_f64(t) for t in s.enc_E]
    for b in (0, 33, w.B - 1):
        ob = s.book(b)
        k = int(first[b].item()) + 2
        want = _oracle_embed(ob.entries[k], s.W_E, encE64, w.heads)
        err = np.abs(E32[b, k].cpu().double().numpy() - want).max()
        assert err <= TOL, (b, k, err)
        assert torch.equal(s.E_h[b, k].cpu(), E32[b, k].cpu().to(w.torch_dtype))

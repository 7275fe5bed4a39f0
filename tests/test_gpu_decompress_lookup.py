"""GPU parity of LZW decompression (Section 2.1, Section 2.3 steps 11-12) and of the mixed-stream
embedding lookup (Figure 2a), through the C ABI, against the CPU oracle.  Integer work: bit-exact."""
import itertools

import numpy as np
import pytest
import torch

from oracle import embedding as oemb, lzw as olzw
from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import synth_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class Session:
    def __init__(self, V, M, cap, B):
        self.V, self.M, self.cap, self.B = V, M, cap, B
        self.cfg = zb.make_config(V, 8, M, cap, B, "fp32", 0, 1, 8)
        self.cb = zb.Codebook(self.cfg, DEV)

    def entries(self, b):
        cons, ln = zb.z2z_codebook_read(self.cb, b)
        st, n = zb.z2z_status(self.cb)
        return [tuple(int(x) for x in cons[k, :int(ln[k])]) for k in range(int(n[b]))], int(st[b])

    def decode(self, code_rows, mode, T_out, pass_lens=True):
        """code_rows: list of B python lists.  Returns (token rows, status list)."""
        B = self.B
        Tc = max(max((len(r) for r in code_rows), default=0), 1)
        codes = np.full((B, Tc), -5, dtype=np.int32)
        for b, r in enumerate(code_rows):
            codes[b, :len(r)] = r
        g_codes = torch.from_numpy(codes).to(DEV)
        g_lens = torch.tensor([len(r) for r in code_rows], dtype=torch.int32, device=DEV) if pass_lens else None
        toks = torch.full((B, max(T_out, 1)), -9, dtype=torch.int32, device=DEV)
        tlen = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        zb.z2z_lzw_decode(self.cb, g_codes, g_lens, mode, toks, tlen)
        st, _ = zb.z2z_status(self.cb)
        toks, tlen = toks.cpu().numpy(), tlen.cpu().numpy()
        rows = [toks[b, :tlen[b]].tolist() for b in range(B)]
        for b in range(B):                                   # nothing written past the reported length
            assert np.all(toks[b, tlen[b]:] == -9)
        return rows, [int(s) for s in st]


def _encode_rows(w, seed, T=None):
    w = w if T is None else w.scaled(T=T)
    tokens = si.make_tokens(w, seed)
    enc = [olzw.encode(tokens[b].tolist(), w.V, w.M, w.cap) for b in range(w.B)]
    return tokens, enc


@pytest.mark.parametrize("name,B,T", [("tiny", 3, 256), ("phi3_mini_head", 8, 2048),
                                      ("long_context", 2, 32768), ("prefill_heavy", 5, 8192)])
def test_replay_decode_is_self_contained_and_rebuilds_the_codebook(name, B, T):
    w = si.WORKLOADS[name].scaled(B=B, T=T)
    tokens, enc = _encode_rows(w, 31)
    s = Session(w.V, w.M, w.cap, w.B)                         # fresh session: empty codebooks
    rows, st = s.decode([e[0] for e in enc], zb.DECODE_REPLAY, T)
    for b in range(B):
        want, ob = olzw.decode(enc[b][0], w.V, w.M, w.cap)
        assert want == tokens[b].tolist()
        assert rows[b] == want
        ents, _ = s.entries(b)
        assert ents == ob.entries == enc[b][2].entries
        assert st[b] & ~zb.ST_CAP_FROZEN == 0
    # the same codes expanded again with the now-resident codebook: same tokens, codebook untouched
    rows2, _ = s.decode([e[0] for e in enc], zb.DECODE_RESIDENT, T)
    assert rows2 == rows
    for b in range(B):
        assert s.entries(b)[0] == enc[b][2].entries


def test_resident_decode_after_gpu_encode_and_steps_ragged_lengths():
    """The session that compressed the prompts and took online updates expands its own stream."""
    w = si.WORKLOADS["tiny"].scaled(B=4, T=700, cap=128)
    tokens = si.make_tokens(w, 33)
    lens = [700, 0, 1, 333]
    s = Session(w.V, w.M, w.cap, w.B)
    g_tok = torch.from_numpy(tokens).to(DEV)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=DEV)
    clen = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    zb.z2z_lzw_encode(s.cb, g_tok, torch.tensor(lens, dtype=torch.int32, device=DEV), codes, clen, None)
    books = []
    streams = []
    for b in range(w.B):
        oc, _, ob = olzw.encode(tokens[b, :lens[b]].tolist(), w.V, w.M, w.cap)
        assert codes[b, :int(clen[b])].cpu().tolist() == oc
        books.append(ob)
        streams.append(list(oc))
    rng = np.random.default_rng(34)
    ne = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    for t in range(40):                                       # generated codes, not a greedy parse
        z = [int(rng.integers(0, w.V + books[b].n())) for b in range(w.B)]
        zb.z2z_lzw_step(s.cb, torch.tensor(z, dtype=torch.int32, device=DEV), None, ne)
        for b in range(w.B):
            assert ne[b].item() == books[b].step(z[b])
            streams[b].append(z[b])
    T_out = max(olzw.base_token_count(books[b], streams[b]) for b in range(w.B))
    rows, st = s.decode(streams, zb.DECODE_RESIDENT, T_out)
    for b in range(w.B):
        want, done = olzw.expand(books[b], streams[b])
        assert done == len(streams[b]) and rows[b] == want
        assert st[b] & (zb.ST_BAD_TOKEN | zb.ST_OUTPUT_TRUNCATED) == 0
    # a fresh session replaying the whole stream (prompt codes + generated codes) agrees
    s2 = Session(w.V, w.M, w.cap, w.B)
    rows2, _ = s2.decode(streams, zb.DECODE_REPLAY, T_out)
    assert rows2 == rows
    for b in range(w.B):
        assert s2.entries(b)[0] == books[b].entries


def test_replay_brute_force_all_code_streams_on_tiny_vocabularies():
    """Every code stream of length <= 5 over ids 0..V+3, legal or not, against the oracle's
    replay: accepted prefix, tokens, codebook and BAD_TOKEN."""
    V, M, cap = 2, 3, 3
    for L in (1, 3, 5):
        allz = list(itertools.product(range(V + 4), repeat=L))
        for s0 in range(0, len(allz), 1024):
            chunk = allz[s0:s0 + 1024]
            s = Session(V, M, cap, len(chunk))
            rows, st = s.decode([list(c) for c in chunk], zb.DECODE_REPLAY, L * M, pass_lens=(L != 3))
            for b, c in enumerate(chunk):
                ob = olzw.Codebook(V, M, cap)
                want = []
                bad = False
                for z in c:
                    ob.step(z)
                    if ob.status & olzw.BAD_TOKEN:
                        bad = True
                        break
                    want.extend(ob.phrase(z))
                assert rows[b] == want, (c, rows[b], want)
                assert bool(st[b] & zb.ST_BAD_TOKEN) == bad, (c, st[b])
                assert s.entries(b)[0] == ob.entries, c


def test_decode_stops_at_bad_codes_and_reports_truncation():
    w = si.WORKLOADS["tiny"].scaled(B=3, T=8000, cap=256)     # > 2 chunks of codes per sequence
    tokens, enc = _encode_rows(w, 35)
    streams = [list(e[0]) for e in enc]
    assert min(len(x) for x in streams) > 4200
    s = Session(w.V, w.M, w.cap, w.B)
    s.decode(streams, zb.DECODE_REPLAY, w.T)                  # make the codebooks resident
    broken = [list(x) for x in streams]
    broken[0][4100] = w.V + w.cap + 7                         # in the third chunk
    broken[1][2048] = -1                                      # first code of the second chunk
    rows, st = s.decode(broken, zb.DECODE_RESIDENT, w.T)
    for b in range(w.B):
        want, done = olzw.expand(enc[b][2], broken[b])
        assert rows[b] == want
        assert bool(st[b] & zb.ST_BAD_TOKEN) == (done < len(broken[b]))
    assert st[2] & zb.ST_BAD_TOKEN == 0
    # output buffer too small: exactly T_out tokens, flag set
    s3 = Session(w.V, w.M, w.cap, w.B)
    rows, st = s3.decode(streams, zb.DECODE_REPLAY, 1000)
    for b in range(w.B):
        assert rows[b] == tokens[b, :1000].tolist()
        assert st[b] & zb.ST_OUTPUT_TRUNCATED
    # empty input
    s4 = Session(w.V, w.M, w.cap, w.B)
    rows, st = s4.decode([[], [], []], zb.DECODE_REPLAY, 8)
    assert rows == [[], [], []] and st == [0, 0, 0]


@pytest.mark.parametrize("dtype,d", [("fp32", 72), ("bf16", 256), ("bf16", 3072)])
def test_embed_lookup_matches_oracle(dtype, d):
    V, M, cap, B = 1000, 3, 64, 4
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    cfg = zb.make_config(V, d, M, cap, B, dtype, 0, 1, 8)
    cb = zb.Codebook(cfg, DEV)
    w = si.WORKLOADS["tiny"].scaled(V=V, B=B, T=300, cap=cap, M=M)
    tokens = si.make_tokens(w, 37)
    g_tok = torch.from_numpy(tokens).to(DEV)
    codes = torch.zeros(B, w.T, dtype=torch.int32, device=DEV)
    clen = torch.zeros(B, dtype=torch.int32, device=DEV)
    zb.z2z_lzw_encode(cb, g_tok, None, codes, clen, None)
    _, n = zb.z2z_status(cb)
    W_E = si.normal_tensor((V, d), 0.05, 38, tdt)
    E_h = si.normal_tensor((B, cap, d), 0.05, 39, tdt)
    h_codes, h_len = codes.cpu().numpy(), clen.cpu().numpy()
    flat, seq = [], []
    for b in range(B):
        flat += h_codes[b, :h_len[b]].tolist()
        seq += [b] * int(h_len[b])
    flat += [V + int(n[1]), -2]                               # two codes that name nothing
    seq += [1, 3]
    out = torch.full((len(flat), d), 7.0, dtype=tdt, device=DEV)
    zb.z2z_embed_lookup(cb, torch.tensor(flat, dtype=torch.int32, device=DEV),
                        torch.tensor(seq, dtype=torch.int32, device=DEV), W_E.to(DEV), E_h.to(DEV), out)
    want, bad = oemb.lookup(flat, seq, W_E.double().numpy(), E_h.double().numpy(), n.tolist())
    assert np.array_equal(out.cpu().double().numpy(), want)  # a copy: exact
    st, _ = zb.z2z_status(cb)
    for b in range(B):
        assert bool(int(st[b]) & zb.ST_BAD_TOKEN) == (b in bad)
    assert sorted(bad) == [1, 3]
    # without row_seq: row r belongs to sequence r
    z = [V, 5, V + 1, 999]
    out2 = torch.zeros(4, d, dtype=tdt, device=DEV)
    zb.z2z_embed_lookup(cb, torch.tensor(z, dtype=torch.int32, device=DEV), None, W_E.to(DEV), E_h.to(DEV), out2)
    want2, _ = oemb.lookup(z, None, W_E.double().numpy(), E_h.double().numpy(), n.tolist())
    assert np.array_equal(out2.cpu().double().numpy(), want2)


def test_upload_rows_copies_pinned_host_memory():
    src = si.normal_tensor((8, 3072), 1.0, 41, torch.bfloat16).pin_memory()
    dst = torch.zeros(8, 3072, dtype=torch.bfloat16, device=DEV)
    zb.z2z_upload_rows(src, dst)
    assert torch.equal(dst.cpu(), src)
    src2 = si.normal_tensor((3, 8), 1.0, 42, torch.float32).pin_memory()     # 96 bytes: a ragged tail of the last block
    dst2 = torch.zeros(3, 8, dtype=torch.float32, device=DEV)
    zb.z2z_upload_rows(src2, dst2)
    zb.z2z_upload_rows(src2[1:2], dst2[0:1])                                  # a view: row 1 over row 0
    assert torch.equal(dst2.cpu()[1:], src2[1:]) and torch.equal(dst2.cpu()[0], src2[1])


def test_teacher_forcing_codes_of_the_benchmark_continue_the_prompt():
    """The benchmark's teacher-forced mode restarts the session from all but the last of the
    prompt's codes and feeds the steps the codes of the generator's continuation.  Held against
    the oracle: those codes are the oracle's codes of the whole stream at the same positions, the
    restarted session holds the oracle's codebook at that point, and after the codes have been
    applied one per step the session decompresses (replayed codes + forced codes) to the
    generator's own tokens."""
    import os
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if root not in sys.path:
        sys.path.insert(0, root)
    import bench
    w = si.WORKLOADS["tiny"].scaled(B=3, T=200, cap=256)
    n_steps = 40
    stream = si.make_tokens(w, 71, T=w.T + n_steps * w.M + 64)
    prompt = np.ascontiguousarray(stream[:, :w.T])
    s = Session(w.V, w.M, w.cap, w.B)
    codes = torch.zeros(w.B, w.T, dtype=torch.int32, device=DEV)
    clen = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    zb.z2z_lzw_encode(s.cb, torch.from_numpy(prompt).to(DEV), None, codes, clen, None)
    forced = bench.forced_codes(zb, w, s.cb, torch.device(DEV), stream, clen, n_steps).cpu().numpy()
    k = (clen.cpu().numpy() - 1).tolist()
    full = [olzw.encode(stream[b].tolist(), w.V, w.M, w.cap) for b in range(w.B)]
    for b in range(w.B):
        want_codes, want_after, _ = full[b]
        assert olzw.encode(prompt[b].tolist(), w.V, w.M, w.cap)[0][:k[b]] == want_codes[:k[b]]
        assert forced[:, b].tolist() == want_codes[k[b]:k[b] + n_steps]
        ents, st = s.entries(b)
        # an encoder that has emitted k codes has created the entry that the k-th code closes; the
        # decoder-side update creates it one code later
        assert st == 0
        assert len(ents) == (want_after[k[b] - 2] if k[b] >= 2 else 0)
        assert ents == full[b][2].entries[:len(ents)]
    new = torch.zeros(w.B, dtype=torch.int32, device=DEV)
    for t in range(n_steps):
        zb.z2z_lzw_step(s.cb, torch.from_numpy(forced[t]).to(DEV), None, new)
    rows = [full[b][0][:k[b] + n_steps] for b in range(w.B)]
    toks, st = s.decode(rows, zb.DECODE_RESIDENT, w.T + n_steps * w.M + 64)
    for b in range(w.B):
        assert st[b] == 0
        assert toks[b] == stream[b, :len(toks[b])].tolist() and len(toks[b]) > w.T - w.M

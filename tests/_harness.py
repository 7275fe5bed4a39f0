"""Test helpers: build the same seeded session on the GPU (through the C ABI binding) and in the
CPU oracle.  Data flows generator -> both sides, and oracle -> GPU (cache forcing); never
GPU -> oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import decode_step as ods
from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import synth_inputs as si

TOL = 2e-2            # stated tolerance for hyper-embeddings and logits (max abs error vs fp64)
GAP = 1e-3            # selections may differ from the oracle only below this top-2 gap


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


class Pair:
    """One workload instantiated on both sides."""

    def __init__(self, w: si.Workload, seed: int, generic_encoder: bool = True, device="cuda:0",
                 tensor_cores: bool = True):
        self.w, self.dev = w, torch.device(device)
        self.tensor_cores = tensor_cores
        self.tokens = si.make_tokens(w, seed)                              # [B, T] int32
        self.W_E, self.W_U = si.make_tables(w, seed)
        self.enc_E = si.make_encoder(w, seed * 3 + 1, generic=generic_encoder)
        self.enc_U = self.enc_E if w.tied else si.make_encoder(w, seed * 3 + 2,
                                                               generic=generic_encoder)
        # --- oracle side (fp64 views of the exact stored values)
        self.oracle = ods.Session(w.V, w.M, w.cap, w.B, w.heads, w.dtype, f64(self.W_E),
                                  f64(self.W_U), [f64(t) for t in self.enc_E],
                                  [f64(t) for t in self.enc_U])
        # --- GPU side
        self.cfg = zb.make_config(w.V, w.d, w.M, w.cap, w.B, w.dtype, w.enc_layers, w.heads,
                                  w.dff, w.tied)
        self.cb = zb.Codebook(self.cfg, device)
        if int(tensor_cores) != 1:
            # 0: CUDA-core kernels as an on-GPU cross-check; 2 + 16 s: CTA-pair logits kernel
            zb.z2z_set_tensor_cores(self.cb, int(tensor_cores))
        self.g_WE = self.W_E.to(self.dev)
        self.g_WU = self.g_WE if w.tied else self.W_U.to(self.dev)
        self.g_encE_t = [t.to(self.dev) for t in self.enc_E]
        self.g_encU_t = self.g_encE_t if w.tied else [t.to(self.dev) for t in self.enc_U]
        self.g_encE = zb.encoder_weights(self.g_encE_t)
        self.g_encU = zb.encoder_weights(self.g_encU_t)
        self.E_h = torch.zeros(w.B, max(w.cap, 1), w.d, dtype=w.torch_dtype, device=self.dev)
        self.U_h = self.E_h if w.tied else torch.zeros_like(self.E_h)
        self.E_f32 = torch.zeros(w.B, max(w.cap, 1), w.d, dtype=torch.float32, device=self.dev)
        self.U_f32 = torch.zeros_like(self.E_f32)

    # -- prefill on both sides, compared ------------------------------------------------------
    def gpu_encode(self, tokens=None, lens=None):
        w = self.w
        tokens = self.tokens if tokens is None else tokens
        B, T = tokens.shape
        g_tok = torch.from_numpy(np.ascontiguousarray(tokens)).to(self.dev)
        g_lens = None if lens is None else torch.tensor(lens, dtype=torch.int32, device=self.dev)
        codes = torch.full((B, max(T, 1)), -7, dtype=torch.int32, device=self.dev)
        after = torch.full((B, max(T, 1)), -7, dtype=torch.int32, device=self.dev)
        code_lens = torch.zeros(B, dtype=torch.int32, device=self.dev)
        zb.z2z_lzw_encode(self.cb, g_tok, g_lens, codes, code_lens, after)
        return codes.cpu().numpy(), code_lens.cpu().numpy(), after.cpu().numpy()

    def gpu_codebook(self, b):
        cons, ln = zb.z2z_codebook_read(self.cb, b)
        st, n = zb.z2z_status(self.cb)
        ents = [tuple(int(x) for x in cons[k, :int(ln[k])]) for k in range(int(n[b]))]
        return ents, cons.numpy(), ln.numpy(), int(st[b]), int(n[b])

    def check_codebooks(self):
        for b in range(self.w.B):
            ents, cons, ln, st, n = self.gpu_codebook(b)
            ob = self.oracle.books[b]
            assert n == ob.n(), (b, n, ob.n())
            assert ents == ob.entries
            assert np.all(cons[n:] == -1) and np.all(ln[n:] == 0)
            for k in range(n):
                assert np.all(cons[k, int(ln[k]):] == -1)
            assert (st & ~zb.ST_CAP_FROZEN) == (ob.status & ~1), (b, st, ob.status)
            assert bool(st & zb.ST_CAP_FROZEN) == (n >= self.w.cap > 0)

    def force_caches_from_oracle(self, b, lo, hi):
        """Overwrite GPU cache rows [lo, hi) of sequence b with the oracle's stored rows."""
        if hi <= lo:
            return
        dt = self.w.torch_dtype
        self.E_h[b, lo:hi] = torch.from_numpy(self.oracle.E_h[b][lo:hi]).to(dt).to(self.dev)
        if not self.w.tied:
            self.U_h[b, lo:hi] = torch.from_numpy(self.oracle.U_h[b][lo:hi]).to(dt).to(self.dev)

    def check_cache_rows(self, b, lo, hi, tol=TOL):
        """fp32 side output vs the oracle's fp64 rows; stored rows == RNE(side output)."""
        if hi <= lo:
            return 0.0
        worst = 0.0
        for side, f32, exact in ((self.E_h, self.E_f32, self.oracle.E_exact),
                                 (self.U_h, self.U_f32, self.oracle.U_exact)):
            got = f32[b, lo:hi].cpu().double().numpy()
            err = float(np.abs(got - exact[b][lo:hi]).max())
            worst = max(worst, err)
            assert err <= tol, f"hyper-embedding error {err} > {tol} (seq {b}, rows {lo}:{hi})"
            assert torch.equal(side[b, lo:hi].cpu(), f32[b, lo:hi].cpu().to(self.w.torch_dtype))
            if self.w.tied:
                break
        return worst

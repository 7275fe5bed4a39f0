"""Pins for oracle/hyper_encoder.py (CPU only, nothing from the CUDA path)."""
import numpy as np
import pytest
import torch

from oracle import hyper_encoder as he
from paper_2506_01084_b200 import synth_inputs as si


def _setup(layers, d=32, M=4, V=50, heads=4, seed=3, generic=True, ffn=1):
    w = si.Workload("t", V=V, d=d, dtype="fp32", B=1, T=8, M=M, cap=8, zipf_s=1.0, copy_p=0.0,
                    seg_min=1, seg_max=1, steps=0, enc_layers=layers, enc_heads=heads,
                    enc_dff=3 * d, enc_ffn=ffn)
    enc = [t.double().numpy() for t in si.make_encoder(w, seed, generic=generic)]
    W, _ = si.make_tables(w, seed)
    return w, enc, W.double().numpy()


def test_zero_layers_is_the_averaging_variant():
    # the parameter-free "averaging" hyper-encoder of the architecture ablation: with pos = 0
    # the output is exactly the mean of the constituent rows (pins gather, padding, pooling)
    w, enc, W = _setup(0)
    enc[0][:] = 0.0
    for e in [(3, 7), (1, 2, 3), (9, 9, 9, 4)]:
        got = he.hyper_embed_one(e, W, enc, w.heads)
        np.testing.assert_allclose(got, W[list(e)].mean(axis=0), rtol=0, atol=1e-15)
    # with pos != 0 it is the mean of (row + pos_i)
    w, enc, W = _setup(0)
    got = he.hyper_embed_one((5, 6, 7), W, enc, w.heads)
    np.testing.assert_allclose(got, (W[[5, 6, 7]] + enc[0][:3]).mean(axis=0), atol=1e-15)


@pytest.mark.parametrize("layers", [1, 2])
def test_against_library_encoder_layer(layers):
    # the textbook pre-LN encoder layer as shipped by the installed PyTorch, fp64, same weights,
    # padded to M with a key-padding mask; pooled over valid positions
    w, enc, W = _setup(layers)
    d, M = w.d, w.M
    mods = []
    for l in range(layers):
        m = torch.nn.TransformerEncoderLayer(d, w.heads, dim_feedforward=w.dff, dropout=0.0,
                                             activation="gelu", batch_first=True,
                                             norm_first=True, dtype=torch.float64)
        t = [torch.from_numpy(a) for a in enc[1 + 12 * l: 13 + 12 * l]]
        with torch.no_grad():
            m.norm1.weight.copy_(t[0]); m.norm1.bias.copy_(t[1])
            m.self_attn.in_proj_weight.copy_(t[2]); m.self_attn.in_proj_bias.copy_(t[3])
            m.self_attn.out_proj.weight.copy_(t[4]); m.self_attn.out_proj.bias.copy_(t[5])
            m.norm2.weight.copy_(t[6]); m.norm2.bias.copy_(t[7])
            m.linear1.weight.copy_(t[8]); m.linear1.bias.copy_(t[9])
            m.linear2.weight.copy_(t[10]); m.linear2.bias.copy_(t[11])
        m.eval()
        mods.append(m)
    entries = [(3, 7), (1, 2, 3), (9, 9, 9, 4), (4, 9, 9, 9)]
    for e in entries:
        L = len(e)
        x = torch.zeros(1, M, d, dtype=torch.float64)
        x[0, :L] = torch.from_numpy(W[list(e)] + enc[0][:L])
        x[0, L:] = 123.0                               # padding garbage must not matter
        mask = torch.zeros(1, M, dtype=torch.bool)
        mask[0, L:] = True
        with torch.no_grad():
            for m in mods:
                # keep torch on its reference path (the fused fast path rewrites padded rows)
                x = m(x, src_key_padding_mask=mask)
        want = x[0, :L].mean(dim=0).numpy()
        got = he.hyper_embed_one(e, W, enc, w.heads)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    # batched form == one-by-one form
    many = he.hyper_embed(entries, W, enc, w.heads)
    for i, e in enumerate(entries):
        np.testing.assert_allclose(many[i], he.hyper_embed_one(e, W, enc, w.heads), atol=1e-13)


@pytest.mark.parametrize("layers", [1, 2])
def test_attention_only_layers_against_library_attention(layers):
    # the "1-attention-layer" variant of the architecture ablation, read as the attention
    # sublayer of the same pre-LN layer: X + MHA(LN1(X)), with the installed PyTorch's
    # multi-head attention (fp64, same weights, key-padding mask) as the library routine
    w, enc, W = _setup(layers, ffn=0)
    d, M = w.d, w.M
    assert enc[1 + 8].shape == (0, d) and enc[1 + 10].shape == (d, 0)
    entries = [(3, 7), (1, 2, 3), (9, 9, 9, 4), (4, 9, 9, 9)]
    for e in entries:
        L = len(e)
        x = torch.zeros(1, M, d, dtype=torch.float64)
        x[0, :L] = torch.from_numpy(W[list(e)] + enc[0][:L])
        x[0, L:] = -77.0
        mask = torch.zeros(1, M, dtype=torch.bool)
        mask[0, L:] = True
        for l in range(layers):
            t = [torch.from_numpy(a) for a in enc[1 + 12 * l: 13 + 12 * l]]
            mha = torch.nn.MultiheadAttention(d, w.heads, dropout=0.0, batch_first=True, dtype=torch.float64)
            with torch.no_grad():
                mha.in_proj_weight.copy_(t[2]); mha.in_proj_bias.copy_(t[3])
                mha.out_proj.weight.copy_(t[4]); mha.out_proj.bias.copy_(t[5])
                a = torch.nn.functional.layer_norm(x, (d,), t[0], t[1], 1e-5)
                x = x + mha(a, a, a, key_padding_mask=mask, need_weights=False)[0]
        want = x[0, :L].mean(dim=0).numpy()
        np.testing.assert_allclose(he.hyper_embed_one(e, W, enc, w.heads), want, rtol=0, atol=1e-12)
    many = he.hyper_embed(entries, W, enc, w.heads)
    for i, e in enumerate(entries):
        np.testing.assert_allclose(many[i], he.hyper_embed_one(e, W, enc, w.heads), atol=1e-13)
    # it is not the full layer: the feed-forward block changes the result
    wf, encf, Wf = _setup(layers, ffn=1)
    assert np.abs(he.hyper_embed_one((1, 2, 3), Wf, encf, w.heads) - many[1]).max() > 1e-4


def test_attention_only_with_zero_output_projection_is_the_mean():
    # Wo = 0, bo = 0: the sublayer adds nothing, so the result is the averaging variant
    w, enc, W = _setup(2, ffn=0)
    for l in range(2):
        enc[1 + 12 * l + 4][:] = 0.0
        enc[1 + 12 * l + 5][:] = 0.0
    got = he.hyper_embed_one((5, 6, 7), W, enc, w.heads)
    np.testing.assert_allclose(got, (W[[5, 6, 7]] + enc[0][:3]).mean(axis=0), atol=1e-15)


def test_order_matters_and_padding_is_inert():
    w, enc, W = _setup(2)
    a = he.hyper_embed_one((3, 7), W, enc, w.heads)
    b = he.hyper_embed_one((7, 3), W, enc, w.heads)
    assert np.abs(a - b).max() > 1e-6                 # "a b" and "b a" must not collide
    # a phrase of length L < M is computed from its L rows only: same answer at any M
    w5, enc5, W5 = _setup(2, M=6)
    enc5[0][:4] = enc[0][:4]
    for i in range(1, len(enc)):
        enc5[i] = enc[i]
    np.testing.assert_allclose(he.hyper_embed_one((3, 7, 1), W, enc5, w.heads),
                               he.hyper_embed_one((3, 7, 1), W, enc, w.heads), atol=0)


def test_gelu_and_layernorm_closed_forms():
    x = np.array([[-1.0, 0.0, 1.0, 2.0]])
    # Phi(1) = 0.841344746..., GELU(1) = 0.841344746, GELU(-1) = -0.158655254
    g = he._gelu(x)
    np.testing.assert_allclose(g[0], [-0.15865525393145707, 0.0, 0.8413447460685429,
                                      1.9544997361036416], atol=1e-15)
    y = he._layer_norm(x, np.ones(4), np.zeros(4))
    assert abs(y.mean()) < 1e-15 and abs((y ** 2).mean() - 1.25 / (1.25 + 1e-5)) < 1e-12

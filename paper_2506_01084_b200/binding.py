"""ctypes binding of the C ABI in include/z2z.h: same names, argument marshalling only.

Every call takes torch tensors (device memory owned by the caller) and forwards raw pointers and
the current CUDA stream.  Nothing is computed here; if the shared library has not been built the
import of the library fails loudly (there is no fallback path).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libz2z.so")

OK = 0
ST_CAP_FROZEN, ST_BAD_TOKEN, ST_TABLE_FULL, ST_WAIT_TIMEOUT, ST_OUTPUT_TRUNCATED, ST_HALF_RANGE = 1, 2, 4, 8, 16, 32
DTYPE_FP32, DTYPE_BF16 = 0, 1
SELECT_ARGMAX, SELECT_GUMBEL = 0, 1
CODE_NONE, CODE_SELECTED = -1, -2
CACHE_EMBED, CACHE_UNEMBED = 0, 1
DECODE_RESIDENT, DECODE_REPLAY = 0, 1

EXPORTS = ["z2z_workspace_bytes", "z2z_codebook_init", "z2z_lzw_encode", "z2z_lzw_step",
           "z2z_hyper_embed", "z2z_dynamic_logits", "z2z_decode_step", "z2z_status",
           "z2z_codebook_read", "z2z_codebook_destroy", "z2z_last_error", "z2z_profile",
           "z2z_profile_read", "z2z_set_tensor_cores", "z2z_logits_static_scratch",
           "z2z_lzw_decode", "z2z_embed_lookup", "z2z_upload_rows", "z2z_sample_filtered",
           "z2z_set_encoder_half_scratch"]


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("V", "d", "M", "cap", "B", "dtype", "enc_layers",
                                         "enc_heads", "enc_dff", "tied")]


class EncoderWeights(C.Structure):
    _fields_ = [("tensors", C.POINTER(C.c_void_p)), ("n_tensors", C.c_int32)]


class Z2ZError(RuntimeError):
    pass


_lib = None


def lib() -> C.CDLL:
    """Load the shared library (once).  Raises if it is missing: build it first with
    ``python -m paper_2506_01084_b200.build``."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise Z2ZError(f"{LIB_PATH} not found: run `python -m paper_2506_01084_b200.build`")
        _lib = C.CDLL(LIB_PATH)
        _lib.z2z_last_error.restype = C.c_char_p
        for name in EXPORTS:
            if name != "z2z_last_error":
                getattr(_lib, name).restype = C.c_int32
    return _lib


def _check(rc: int):
    if rc != OK:
        raise Z2ZError(f"z2z error {rc}: {lib().z2z_last_error().decode()}")


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return C.c_void_p(0)
    assert t.is_contiguous(), "tensors passed to the ABI must be contiguous"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(V, d, M, cap, B, dtype, enc_layers, enc_heads, enc_dff, tied=0) -> Config:
    if dtype in ("fp32", torch.float32):
        dt = DTYPE_FP32
    elif dtype in ("bf16", torch.bfloat16):
        dt = DTYPE_BF16
    else:
        dt = int(dtype)
    return Config(V, d, M, cap, B, dt, enc_layers, enc_heads, enc_dff, tied)


def encoder_weights(tensors: Sequence[torch.Tensor]) -> EncoderWeights:
    """HOST array of DEVICE pointers in ABI order.  The returned struct keeps the array alive."""
    arr = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    ew = EncoderWeights(C.cast(arr, C.POINTER(C.c_void_p)), len(tensors))
    ew._keep = (arr, list(tensors))
    return ew


def z2z_workspace_bytes(cfg: Config) -> int:
    out = C.c_size_t(0)
    _check(lib().z2z_workspace_bytes(C.byref(cfg), C.byref(out)))
    return out.value


class Codebook:
    """Owns the opaque handle; the workspace tensor is allocated by the caller side (torch)."""

    def __init__(self, cfg: Config, device="cuda:0"):
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = z2z_workspace_bytes(cfg)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + off
        self._ws_bytes = nbytes
        self.handle = C.c_void_p(0)
        z2z_codebook_init(self)

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.z2z_codebook_destroy(self.handle)
                self.handle = C.c_void_p(0)
        except Exception:
            pass


def z2z_codebook_init(cb: Codebook):
    _check(lib().z2z_codebook_init(C.byref(cb.handle), C.byref(cb.cfg), C.c_void_p(cb._ws_ptr),
                                   C.c_size_t(cb._ws_bytes), _stream()))


def z2z_lzw_encode(cb: Codebook, tokens: torch.Tensor, lens: Optional[torch.Tensor],
                   codes: torch.Tensor, code_lens: torch.Tensor,
                   entries_after: Optional[torch.Tensor] = None):
    T_max = tokens.shape[1] if tokens.dim() == 2 else 0
    _check(lib().z2z_lzw_encode(cb.handle, _ptr(tokens), _ptr(lens), C.c_int32(T_max), _ptr(codes),
                                _ptr(code_lens), _ptr(entries_after), _stream()))


def z2z_lzw_step(cb: Codebook, new_codes: torch.Tensor, active: Optional[torch.Tensor],
                 new_entry: Optional[torch.Tensor]):
    _check(lib().z2z_lzw_step(cb.handle, _ptr(new_codes), _ptr(active), _ptr(new_entry), _stream()))


def z2z_hyper_embed(cb: Codebook, which: int, table: torch.Tensor, enc: EncoderWeights,
                    first: Optional[torch.Tensor], count: Optional[torch.Tensor], max_entries: int,
                    cache: torch.Tensor, cache_f32: Optional[torch.Tensor] = None):
    _check(lib().z2z_hyper_embed(cb.handle, C.c_int32(which), _ptr(table), C.byref(enc),
                                 _ptr(first), _ptr(count), C.c_int32(max_entries), _ptr(cache),
                                 _ptr(cache_f32), _stream()))


def z2z_dynamic_logits(cb: Codebook, hidden: torch.Tensor, row_seq: Optional[torch.Tensor],
                       row_nvis: Optional[torch.Tensor], W_U: torch.Tensor, U_h: torch.Tensor,
                       select: int, temperature: float, seed: int, step: int,
                       targets: Optional[torch.Tensor], lse: Optional[torch.Tensor],
                       argmax: Optional[torch.Tensor], max_logit: Optional[torch.Tensor],
                       sample: Optional[torch.Tensor] = None,
                       target_logit: Optional[torch.Tensor] = None,
                       logits_debug: Optional[torch.Tensor] = None):
    N = hidden.shape[0]
    _check(lib().z2z_dynamic_logits(cb.handle, _ptr(hidden), C.c_int32(N), _ptr(row_seq),
                                    _ptr(row_nvis), _ptr(W_U), _ptr(U_h), C.c_int32(select),
                                    C.c_float(temperature), C.c_uint64(seed), C.c_uint64(step),
                                    _ptr(targets), _ptr(lse), _ptr(argmax), _ptr(max_logit),
                                    _ptr(sample), _ptr(target_logit), _ptr(logits_debug), _stream()))


def z2z_decode_step(cb: Codebook, hidden: torch.Tensor, W_E: torch.Tensor, W_U: torch.Tensor,
                    enc_E: EncoderWeights, enc_U: EncoderWeights, E_h: torch.Tensor,
                    U_h: torch.Tensor, select: int, temperature: float, seed: int, step: int,
                    forced: Optional[torch.Tensor], next_codes: torch.Tensor,
                    selected: Optional[torch.Tensor], lse: Optional[torch.Tensor],
                    new_entry: Optional[torch.Tensor] = None,
                    E_h_f32: Optional[torch.Tensor] = None, U_h_f32: Optional[torch.Tensor] = None,
                    next_embed: Optional[torch.Tensor] = None):
    _check(lib().z2z_decode_step(cb.handle, _ptr(hidden), _ptr(W_E), _ptr(W_U), C.byref(enc_E),
                                 C.byref(enc_U), _ptr(E_h), _ptr(U_h), C.c_int32(select),
                                 C.c_float(temperature), C.c_uint64(seed), C.c_uint64(step),
                                 _ptr(forced), _ptr(next_codes), _ptr(selected), _ptr(lse),
                                 _ptr(new_entry), _ptr(E_h_f32), _ptr(U_h_f32), _ptr(next_embed), _stream()))


def z2z_lzw_decode(cb: Codebook, codes: torch.Tensor, code_lens: Optional[torch.Tensor], mode: int,
                   tokens: torch.Tensor, token_lens: torch.Tensor):
    """codes [B, Tc_max] int32 -> tokens [B, T_out_max] int32, token_lens [B] (device tensors)."""
    Tc_max = codes.shape[1] if codes.dim() == 2 else 0
    T_out = tokens.shape[1] if tokens.dim() == 2 else 0
    _check(lib().z2z_lzw_decode(cb.handle, _ptr(codes), _ptr(code_lens), C.c_int32(Tc_max),
                                C.c_int32(mode), _ptr(tokens), _ptr(token_lens), C.c_int32(T_out),
                                _stream()))


def z2z_embed_lookup(cb: Codebook, codes: torch.Tensor, row_seq: Optional[torch.Tensor],
                     W_E: torch.Tensor, E_h: torch.Tensor, out: torch.Tensor):
    """codes [N] int32 -> out [N, d]: W_E rows for base tokens, cached E_h rows for hypertokens."""
    _check(lib().z2z_embed_lookup(cb.handle, _ptr(codes), C.c_int32(codes.numel()), _ptr(row_seq),
                                  _ptr(W_E), _ptr(E_h), _ptr(out), _stream()))


def z2z_sample_filtered(logits: torch.Tensor, n_cols: torch.Tensor, top_k: int, top_p: float, temperature: float,
                        seed: int, step: int, choice: torch.Tensor, kept: Optional[torch.Tensor] = None,
                        row_base: int = 0):
    """logits [N, ld] fp32 (device), n_cols [N] int32 -> choice [N] int32 (and kept [N] int32)."""
    assert logits.dtype == torch.float32 and logits.dim() == 2
    _check(lib().z2z_sample_filtered(_ptr(logits), C.c_int32(logits.shape[0]), C.c_int64(logits.stride(0)),
                                     _ptr(n_cols), C.c_int32(top_k), C.c_float(top_p), C.c_float(temperature),
                                     C.c_uint64(seed), C.c_uint64(step), C.c_int32(row_base), _ptr(choice), _ptr(kept),
                                     _stream()))


def z2z_upload_rows(src_pinned: torch.Tensor, dst: torch.Tensor):
    """Pinned host tensor -> device tensor of the same size, by a kernel (see z2z.h)."""
    nbytes = src_pinned.numel() * src_pinned.element_size()
    assert src_pinned.is_pinned() and nbytes == dst.numel() * dst.element_size()
    _check(lib().z2z_upload_rows(_ptr(src_pinned), _ptr(dst), C.c_size_t(nbytes), _stream()))


def z2z_status(cb: Codebook):
    """(status bits [B], hypertoken counts [B]) as host int32 tensors; waits for the stream."""
    B = cb.cfg.B
    st = torch.empty(B, dtype=torch.int32)
    n = torch.empty(B, dtype=torch.int32)
    _check(lib().z2z_status(cb.handle, _ptr(st), _ptr(n), _stream()))
    return st, n


def z2z_codebook_read(cb: Codebook, b: int):
    """Codebook of sequence b on the host: (constituents [cap, M] int32, lengths [cap] int32)."""
    cons = torch.empty(cb.cfg.cap, cb.cfg.M, dtype=torch.int32)
    ln = torch.empty(cb.cfg.cap, dtype=torch.int32)
    _check(lib().z2z_codebook_read(cb.handle, C.c_int32(b), _ptr(cons), _ptr(ln), _stream()))
    return cons, ln


PROFILE_CLASSES = ["logits", "logits_merge", "lzw", "encoder_gemm", "encoder_other"]


def z2z_profile(cb: Codebook, enable: bool):
    _check(lib().z2z_profile(cb.handle, C.c_int32(1 if enable else 0)))


def z2z_profile_read(cb: Codebook):
    """({class: milliseconds}, {class: launches}) since the last read; waits for the stream."""
    n = len(PROFILE_CLASSES)
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _check(lib().z2z_profile_read(cb.handle, C.c_int32(n), ms, cnt, _stream()))
    return ({k: ms[i] for i, k in enumerate(PROFILE_CLASSES)},
            {k: int(cnt[i]) for i, k in enumerate(PROFILE_CLASSES)})


def z2z_set_tensor_cores(cb: Codebook, enable):
    """0 / False: CUDA-core kernels; 1 / True: tensor-core kernels chosen by shape;
    2 + 16 * s: the CTA-pair logits kernel for every z2z_dynamic_logits call, with s column strips
    (0: chosen by shape)."""
    _check(lib().z2z_set_tensor_cores(cb.handle, C.c_int32(int(enable))))


def encoder_half_bytes(cfg: Config) -> int:
    """Bytes of scratch z2z_set_encoder_half_scratch needs for this configuration."""
    return 2 * cfg.enc_layers * (4 * cfg.d * cfg.d + 2 * cfg.d * cfg.enc_dff)


def z2z_set_encoder_half_scratch(cb: Codebook, scratch: Optional[torch.Tensor]):
    """Lend device memory (a uint8 tensor, 256-byte aligned) for fp16 copies of one encoder's
    linear-layer weights: long prompt-sized z2z_hyper_embed calls then run one tensor-core pass per
    k-step.  None returns to the two-part form.  The handle keeps a reference to the tensor."""
    cb._half_scratch = scratch
    nbytes = 0 if scratch is None else scratch.numel() * scratch.element_size()
    _check(lib().z2z_set_encoder_half_scratch(cb.handle, _ptr(scratch), C.c_size_t(nbytes)))


def z2z_logits_static_scratch(hidden: torch.Tensor, row_seq: Optional[torch.Tensor],
                              n_hyper: torch.Tensor, W_U: torch.Tensor,
                              U_h: Optional[torch.Tensor], cap: int,
                              lse: Optional[torch.Tensor], argmax: Optional[torch.Tensor],
                              max_logit: Optional[torch.Tensor]):
    """Joint logits + LSE / argmax / maximum without a session handle or workspace: for callers
    that cannot allocate device memory.  The partial reductions live in a fixed 2 MiB array
    inside the library (at most 1024 hidden rows per call).  ``n_hyper`` is a device int32 tensor
    [B] with the visible hypertokens of each sequence.  Calls that overlap on one GPU race on the
    shared array; the first call on a device should be made outside stream capture."""
    N, d = hidden.shape
    V = W_U.shape[0]
    B = n_hyper.shape[0]
    dt = DTYPE_FP32 if hidden.dtype == torch.float32 else DTYPE_BF16
    _check(lib().z2z_logits_static_scratch(_ptr(hidden), C.c_int32(N), _ptr(row_seq),
                                           _ptr(n_hyper), _ptr(W_U), _ptr(U_h), C.c_int32(V),
                                           C.c_int32(d), C.c_int32(B), C.c_int32(cap),
                                           C.c_int32(dt), _ptr(lse), _ptr(argmax),
                                           _ptr(max_logit), _stream()))

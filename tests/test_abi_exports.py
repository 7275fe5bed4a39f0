"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares.
No compute call is made here."""
import ctypes
import os
import re

from paper_2506_01084_b200 import binding as zb
from paper_2506_01084_b200 import build as zbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "z2z.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(z2z_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = zbuild.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"z2z_codebook_init", "z2z_lzw_encode", "z2z_lzw_step", "z2z_hyper_embed",
            "z2z_dynamic_logits", "z2z_decode_step"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in z2z.h but not exported"
    assert sorted(zb.EXPORTS) == names          # the binding wraps exactly the declared calls


def test_host_side_argument_checks_need_no_gpu():
    lib = zb.lib()
    out = ctypes.c_size_t(0)
    bad = zb.make_config(512, 60, 3, 256, 1, "fp32", 2, 4, 256)        # d % 8 != 0
    assert lib.z2z_workspace_bytes(ctypes.byref(bad), ctypes.byref(out)) == -1
    assert b"d %" in lib.z2z_last_error()
    bad = zb.make_config(512, 64, 9, 256, 1, "fp32", 2, 4, 256)         # M too large
    assert lib.z2z_workspace_bytes(ctypes.byref(bad), ctypes.byref(out)) == -1
    bad = zb.make_config(1 << 24, 64, 3, 256, 1, "fp32", 2, 4, 256)     # ids do not fit
    assert lib.z2z_workspace_bytes(ctypes.byref(bad), ctypes.byref(out)) == -1
    ok = zb.make_config(512, 64, 3, 256, 1, "fp32", 2, 4, 256)
    assert lib.z2z_workspace_bytes(ctypes.byref(ok), ctypes.byref(out)) == 0 and out.value > 0
    full = out.value
    # feed-forward width 0 = attention-only layers: accepted, and needs less scratch; 4 is no width
    ok = zb.make_config(512, 64, 3, 256, 1, "fp32", 2, 4, 0)
    assert lib.z2z_workspace_bytes(ctypes.byref(ok), ctypes.byref(out)) == 0 and 0 < out.value < full
    bad = zb.make_config(512, 64, 3, 256, 1, "fp32", 2, 4, 4)
    assert lib.z2z_workspace_bytes(ctypes.byref(bad), ctypes.byref(out)) == -1
    # a NULL handle is rejected, not dereferenced
    assert lib.z2z_lzw_step(None, None, None, None, None) == -1
    assert lib.z2z_lzw_decode(None, None, None, 0, 0, None, None, 0, None) == -1
    assert lib.z2z_embed_lookup(None, None, 0, None, None, None, None, None) == -1
    assert lib.z2z_upload_rows(None, None, ctypes.c_size_t(16), None) == -1
    assert lib.z2z_upload_rows(None, None, ctypes.c_size_t(0), None) == 0
    assert lib.z2z_sample_filtered(None, 4, ctypes.c_int64(8), None, 0, ctypes.c_float(1.0), ctypes.c_float(1.0),
                                   ctypes.c_uint64(0), ctypes.c_uint64(0), 0, None, None, None) == -1
    assert lib.z2z_codebook_destroy(None) == 0

"""Host-only checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before touching the device.  No compute call is made here."""
import ctypes
import os
import re

import pytest

import paper_2607_02980_b200 as hils
from paper_2607_02980_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hils.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hils_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = hils.load_library()
    names = declared_functions()
    assert set(binding.EXPORTS) <= set(names)
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), "libhils.so does not export %s" % n


def test_version_and_status_strings():
    assert hils.version().count(".") == 1
    assert hils.status_string(0) == "ok"
    for code in range(-7, 0):
        assert hils.status_string(code) not in ("ok", "unknown status")
    assert hils.status_string(-99) == "unknown status"


def good(**kw):
    base = dict(B=1, Hq=8, Hkv=2, Hl=2, L=1024, T_max=1024, C=16, d=128, chunk_size=64, top_k=4,
                window=1, scale=0.0, dtype=binding.HILS_BF16, impl="generic")
    base.update(kw)
    return hils.make_params(**base)


def test_workspace_bytes_valid_and_invalid():
    assert hils.workspace_bytes(good(), False) >= 256
    assert hils.workspace_bytes(good(), True) >= 256
    assert hils.host_arena_bytes(good(), False) > 1024 * 128 * 2 * 8
    for bad in (good(Hq=7), good(Hl=3), good(d=0), good(top_k=0), good(window=0), good(dtype=5),
                good(chunk_size=0), good(C=3), good(T_max=512)):
        assert hils.workspace_bytes(bad, False) == 0
    assert hils.workspace_bytes(good(T_max=0), True) == 0
    # shapes the generic kernels do not take
    assert hils.workspace_bytes(good(d=48), False) == 0
    assert hils.workspace_bytes(good(top_k=129, C=16), False) == 0


def call_prefill(p, q=256, k=256, v=256, lm=256, out=256, lse=256, sel=256, ws=256, ws_bytes=1 << 20):
    lib = hils.load_library()
    vp = ctypes.c_void_p
    return lib.hils_prefill(ctypes.byref(p), vp(q), vp(k), vp(v), vp(lm), None, vp(out), vp(lse), vp(sel),
                            vp(ws), ws_bytes, None)


def test_argument_errors_are_returned_before_any_launch():
    """Fake (never dereferenced) pointers: every call must fail on the host with the right code."""
    lib = hils.load_library()
    assert call_prefill(good(Hq=7)) == -1
    assert call_prefill(good(), q=0) == -1
    assert call_prefill(good(), sel=0) == -1
    assert call_prefill(good(), q=264) == -3
    assert call_prefill(good(), lse=258) == -3
    assert call_prefill(good(), ws=0) == -4
    assert call_prefill(good(), ws_bytes=16) == -4
    assert call_prefill(good(d=48)) == -2
    assert call_prefill(good(impl="fast", dtype=binding.HILS_F32)) == -2
    # the packed query-major kernel: bf16, d = 128, four query heads per KV head, top_k <= 32, prefill only
    assert call_prefill(good(impl="packed", dtype=binding.HILS_F32)) == -2
    assert call_prefill(good(impl="packed", Hq=4)) == -2
    assert call_prefill(good(impl="packed", top_k=33, C=64, L=4096, T_max=4096)) == -2
    assert hils.workspace_bytes(good(impl="packed"), False) >= 256
    assert hils.workspace_bytes(good(impl="packed"), True) == 0
    assert lib.hils_prefill(None, None, None, None, None, None, None, None, None, None, 0, None) == -1
    vp = ctypes.c_void_p
    p = good()
    assert lib.hils_decode(ctypes.byref(p), vp(256), vp(256), vp(256), vp(256), None, None, vp(256), vp(256),
                           vp(256), vp(256), 1 << 20, None) == -1          # seq_lens missing
    assert lib.hils_poll_status(None, None) == -1
    assert lib.hils_prefill_host(ctypes.byref(p), vp(256), vp(256), vp(256), vp(256), None, vp(256), vp(256),
                                 vp(256), None, 0, None) == -4
    assert hils.last_launch_count() == 0


def test_binding_rejects_wrong_tensors():
    import torch
    q = torch.zeros(1, 8, 128, 128)
    with pytest.raises((ValueError, TypeError)):
        hils.hils_prefill(q, q, q, q, 64, 4)            # host tensors, mismatched shapes

"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the
header declares, sizes workspaces sensibly and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

from paper_2605_08632_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(cat_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    L = B.lib()
    declared = _declared_symbols()
    assert {"cat_loss_fwd", "cat_loss_bwd", "cat_loss_workspace_bytes", "cat_status_string"} <= declared
    for name in declared:
        assert hasattr(L, name), name


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.cat_shape) == 64
    assert ctypes.sizeof(B.cat_stats) == 32


def test_status_strings():
    for code in range(0, -9, -1):
        assert B.cat_status_string(code) not in ("", "unknown status")
    assert B.cat_status_string(-99) == "unknown status"


def test_workspace_sizes():
    s = B.make_shape(16384, 2048, 128256, 8, B.CAT_BF16)
    fwd, bwd = B.cat_loss_workspace_bytes(s, 0), B.cat_loss_workspace_bytes(s, 1)
    logits_bytes = 16384 * 128256 * 2
    assert 0 < fwd < 64 << 20
    assert 0 < bwd < 0.6 * logits_bytes          # one bounded slab, never the T x V matrix
    big = B.make_shape(131072, 3072, 128256, 32, B.CAT_BF16)
    assert B.cat_loss_workspace_bytes(big, 1) < 0.15 * (131072 * 128256 * 2)
    capped = B.make_shape(16384, 2048, 128256, 8, B.CAT_BF16, slab_mib=256)
    assert B.cat_loss_workspace_bytes(capped, 1) < (256 << 20) + 16384 * 2048 * 4 + (1 << 20)
    fused = B.cat_loss_workspace_bytes(s, 2)
    assert 0 < fused < 0.62 * logits_bytes        # one slab of logits, at least two slabs per batch
    assert B.cat_loss_workspace_bytes(big, 2) < 0.1 * (131072 * 128256 * 2)
    conf_ws = B.cat_loss_workspace_bytes(s, 3)       # cat_conf_fwd: forward scratch + O(T)
    assert fwd <= conf_ws < 2 * fwd + (1 << 20) and B.cat_loss_workspace_bytes(s, 4) == 0
    assert B.cat_loss_launch_count(s, 3) == 3
    assert B.cat_loss_launch_count(s, 0) == 3 and B.cat_loss_launch_count(s, 1) == 7
    assert B.cat_loss_launch_count(s, 2) == 1 + 2 * 6 + 1


@pytest.mark.parametrize("kw,code", [
    (dict(T=0), -2), (dict(T=12, K=8), -2), (dict(K=0), -2), (dict(ldH=100), -2), (dict(in_dtype=7), -3),
    (dict(in_dtype=B.CAT_F32, dW_dtype=B.CAT_BF16), -3), (dict(d=132, ldH=132, ldW=132), -4),
])
def test_bad_shapes_are_rejected_on_the_host(kw, code):
    base = dict(T=64, d=128, V=512, K=8, in_dtype=B.CAT_BF16, dW_dtype=B.CAT_F32, ldH=None, ldW=None)
    base.update(kw)
    s = B.make_shape(**base)
    assert B.cat_loss_workspace_bytes(s, 0) == 0
    L = B.lib()
    fake = ctypes.c_void_p(4096)    # never dereferenced: validation fails first
    rc = L.cat_loss_fwd(ctypes.byref(s), fake, fake, fake, None, None, fake, fake, fake, fake, None, fake, 1 << 30, None)
    assert rc == code
    rc = L.cat_loss_bwd(ctypes.byref(s), fake, fake, fake, None, fake, fake, None, fake, fake, 0, fake, 1 << 30, None)
    assert rc == code


def test_null_alignment_and_workspace_errors():
    L = B.lib()
    s = B.make_shape(64, 128, 512, 8, B.CAT_BF16)
    ok = ctypes.c_void_p(4096)
    need = B.cat_loss_workspace_bytes(s, 0)
    assert L.cat_loss_fwd(ctypes.byref(s), None, ok, ok, None, None, ok, ok, ok, ok, None, ok, need, None) == -1
    assert L.cat_loss_fwd(ctypes.byref(s), ctypes.c_void_p(4098), ok, ok, None, None, ok, ok, ok, ok, None, ok, need, None) == -4
    assert L.cat_loss_fwd(ctypes.byref(s), ok, ok, ok, None, None, ok, ok, ok, ok, None, ok, need - 1, None) == -5
    assert L.cat_loss_fwd(ctypes.byref(s), ok, ok, ok, None, None, ok, ok, ok, ok, None, None, need, None) == -5
    assert L.cat_loss_bwd(ctypes.byref(s), ok, ok, ok, None, ok, ok, None, ok, ok, 0, ok, 16, None) == -5
    assert L.cat_loss_bwd(ctypes.byref(s), ok, ok, ok, None, None, ok, None, ok, ok, 0, ok, 1 << 30, None) == -1

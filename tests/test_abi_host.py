"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its host-side
argument validation answers without touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2605_18753_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_18753_b200 import build
    build.build()
    return B.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "dash_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dash_attn_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 13 and set(names) == set(B.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_debug_library_exports_the_same_symbols_and_swaps_in_and_out(lib):
    from paper_2605_18753_b200 import build
    build.build(debug=True)
    assert os.path.exists(B.DEBUG_LIB_PATH)
    before = B.LIB_PATH
    with B.use_debug_library():
        assert B.LIB_PATH == B.DEBUG_LIB_PATH
        dbg = B.lib()
        for n in _declared():
            assert hasattr(dbg, n), n
        # host-side validation is the same code
        assert dbg.dash_attn_workspace_bytes(ctypes.byref(_p())) == lib.dash_attn_workspace_bytes(ctypes.byref(_p()))
    assert B.LIB_PATH == before and B.lib() is lib


def test_params_struct_matches_header_layout():
    assert ctypes.sizeof(B.DashParams) == 4 * 14 + 8 + 8 * 12
    assert B.DashParams.q_stride.offset == 64


def _p(**kw):
    base = dict(batch=1, seq_q=8192, seq_kv=8192, h_q=32, h_kv=8, head_dim=128, block=64, dtype=B.DASH_BF16, alpha=1.5)
    base.update(kw)
    return B.make_params(**base)


def test_workspace_and_list_geometry(lib):
    p = _p()
    assert B.dash_attn_workspace_bytes(p) > 0
    n, Bk = 8192, 64
    c = n // Bk
    per_head = Bk * c * (c - 1) // 2
    assert B.dash_attn_list_capacity(p) == 8 * per_head
    assert B.dash_attn_list_offset(p, 0, 0, 0) == 0
    assert B.dash_attn_list_offset(p, 0, 0, 64) == 0            # first row with a candidate
    assert B.dash_attn_list_offset(p, 0, 0, 65) == 1
    assert B.dash_attn_list_offset(p, 0, 0, 128) == 64
    assert B.dash_attn_list_offset(p, 0, 3, 130) == 3 * per_head + 64 + 2 * 2
    assert B.dash_attn_list_offset(p, 0, 8, 0) == -1
    # ragged length: rows of the incomplete tail chunk see every complete chunk
    q = _p(seq_q=200, seq_kv=200)
    assert B.dash_attn_list_capacity(q) == 8 * (64 * 3 * 2 // 2 + 8 * 3)
    # decode: one row per (batch, KV head) with room for every complete chunk
    d = _p(batch=16, seq_q=1, seq_kv=131072)
    assert B.dash_attn_list_capacity(d) == 16 * 8 * 2048
    assert B.dash_attn_list_offset(d, 2, 1, 0) == (2 * 8 + 1) * 2048


@pytest.mark.parametrize("kw,code", [
    (dict(h_q=30), -1), (dict(alpha=1.0), -1), (dict(sigma=0.0), -1), (dict(gamma=-1.0), -1),
    (dict(seq_q=100), -1), (dict(head_dim=96), -2), (dict(block=48), -2), (dict(causal=2), -1), (dict(causal=0, local_blocks=1), -1),
    (dict(causal=0, seq_q=1), -2),
    (dict(h_q=24, h_kv=8), -2), (dict(dtype=7), -1), (dict(batch=0), -1), (dict(local_blocks=-1), -1),
])
def test_invalid_parameters_are_rejected_on_the_host(lib, kw, code):
    p = _p(**kw)
    assert B.dash_attn_workspace_bytes(p) == 0
    rc = lib.dash_attn_block_summaries(ctypes.byref(p), 16, None, 0, None, 0, -1, 16, None)
    assert rc == code


def test_local_window_changes_no_size(lib):
    """The window chunks are list entries like the routed ones: same workspace, same list geometry."""
    a, b = _p(), _p(local_blocks=1)
    assert B.dash_attn_workspace_bytes(a) == B.dash_attn_workspace_bytes(b) > 0
    assert B.dash_attn_list_capacity(a) == B.dash_attn_list_capacity(b)
    assert B.dash_attn_list_offset(a, 0, 3, 130) == B.dash_attn_list_offset(b, 0, 3, 130)


def test_non_causal_list_geometry(lib):
    """Without the causal mask every row has all T_s complete chunks as candidates: fixed-size list regions."""
    p = _p(seq_q=200, seq_kv=200, causal=0)
    assert B.dash_attn_list_capacity(p) == 8 * 200 * 3
    assert B.dash_attn_list_offset(p, 0, 2, 7) == 2 * 600 + 21
    assert B.dash_attn_workspace_bytes(p) > 0


def test_null_and_misaligned_pointers_and_short_workspace(lib):
    p = _p()
    assert lib.dash_attn_block_summaries(ctypes.byref(p), None, None, 0, None, 0, -1, 16, None) == -1
    assert lib.dash_attn_block_summaries(ctypes.byref(p), 24, None, 0, None, 0, -1, 16, None) == -1   # not 16-byte aligned
    assert lib.dash_attn_block_summaries(ctypes.byref(p), 16, None, 0, None, 0, 500, 16, None) == -1  # past T_s
    need = B.dash_attn_workspace_bytes(p)
    args = [ctypes.byref(p)] + [256] * 7
    assert lib.dash_attn_attend_prefill(*args, need - 1, None) == -3
    assert lib.dash_attn_attend_prefill(ctypes.byref(p), 256, 256, 256, 256, 256, 256, 128, need, None) == -3
    assert lib.dash_attn_fwd_decode(ctypes.byref(p), 256, 256, 256, 256, None, 256, 256, need, None) == -1  # not a decode shape
    bad = _p()
    bad.struct_size = 8
    assert B.dash_attn_workspace_bytes(bad) == 0
    bad = _p(k_stride=(8192 * 1024, 1023, 128))
    assert B.dash_attn_workspace_bytes(bad) == 0


def test_strerror(lib):
    assert B.strerror(0) == "ok" and "workspace" in B.strerror(-3) and "wait" in B.strerror(-7)

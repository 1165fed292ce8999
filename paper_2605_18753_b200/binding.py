"""ctypes binding of libdash_attn.so: argument marshalling only, every computation runs in the CUDA library.

Function names mirror the C ABI (include/dash_attn.h).  Tensors are torch CUDA tensors used purely as
device buffers; launches go to torch's current stream.  There is no fallback: if the shared library is
missing or cannot be loaded, every call raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_float, c_int32, c_int64, c_size_t, c_uint32, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdash_attn.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libdash_attn_debug.so")    # same library with bounds checks compiled in

DASH_F32, DASH_BF16 = 0, 1
DASH_OK = 0
STATUS = {0: "DASH_OK", -1: "DASH_ERR_INVALID_ARG", -2: "DASH_ERR_UNSUPPORTED", -3: "DASH_ERR_WORKSPACE",
          -4: "DASH_ERR_CAPACITY", -5: "DASH_ERR_CUDA", -6: "DASH_ERR_ARCH", -7: "DASH_ERR_TIMEOUT",
          -8: "DASH_ERR_TOO_LARGE"}

EXPORTS = [
    "dash_attn_workspace_bytes", "dash_attn_list_capacity", "dash_attn_list_offset",
    "dash_attn_block_summaries", "dash_attn_select", "dash_attn_attend_prefill", "dash_attn_attend_decode",
    "dash_attn_attend_decode_static", "dash_attn_bwd_attend_prefill",
    "dash_attn_bwd_workspace_bytes", "dash_attn_bwd_attend_prefill_tc",
    "dash_attn_block_summaries_paged", "dash_attn_fwd_decode_paged",
    "dash_attn_bwd_select_prefill", "dash_attn_bwd_block_summaries",
    "dash_attn_fwd_prefill", "dash_attn_fwd_decode", "dash_attn_reset_status", "dash_attn_last_status",
    "dash_attn_launch_count", "dash_attn_strerror", "dash_attn_test_hooks",
]


class DashError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)} ({strerror(code)})")


class DashParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", c_uint32), ("batch", c_int32), ("seq_q", c_int32), ("seq_kv", c_int32),
        ("h_q", c_int32), ("h_kv", c_int32), ("head_dim", c_int32), ("block", c_int32),
        ("dtype", c_int32), ("causal", c_int32), ("alpha", c_float), ("gamma", c_float), ("sigma", c_float),
        ("local_blocks", c_int32), ("q_to_kv", POINTER(c_int32)),
        ("q_stride", c_int64 * 3), ("k_stride", c_int64 * 3), ("v_stride", c_int64 * 3), ("o_stride", c_int64 * 3),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_18753_b200.build`; "
                               "the DashAttention path has no CPU or PyTorch fallback")
        L = ctypes.CDLL(LIB_PATH)
        P = POINTER(DashParams)
        L.dash_attn_workspace_bytes.restype = c_size_t
        L.dash_attn_workspace_bytes.argtypes = [P]
        L.dash_attn_list_capacity.restype = c_int64
        L.dash_attn_list_capacity.argtypes = [P]
        L.dash_attn_list_offset.restype = c_int64
        L.dash_attn_list_offset.argtypes = [P, c_int32, c_int32, c_int32]
        L.dash_attn_block_summaries.restype = ctypes.c_int
        L.dash_attn_block_summaries.argtypes = [P, c_void_p, c_void_p, c_int64, c_void_p, c_int32, c_int32, c_void_p, c_void_p]
        L.dash_attn_select.restype = ctypes.c_int
        L.dash_attn_select.argtypes = [P] + [c_void_p] * 9 + [c_size_t, c_void_p]
        L.dash_attn_attend_prefill.restype = ctypes.c_int
        L.dash_attn_attend_prefill.argtypes = [P] + [c_void_p] * 7 + [c_size_t, c_void_p]
        L.dash_attn_attend_decode.restype = ctypes.c_int
        L.dash_attn_attend_decode.argtypes = [P] + [c_void_p] * 9 + [c_size_t, c_void_p]
        L.dash_attn_attend_decode_static.restype = ctypes.c_int
        L.dash_attn_attend_decode_static.argtypes = [P] + [c_void_p] * 9
        L.dash_attn_bwd_attend_prefill.restype = ctypes.c_int
        L.dash_attn_bwd_attend_prefill.argtypes = [P] + [c_void_p] * 11
        L.dash_attn_bwd_workspace_bytes.restype = c_size_t
        L.dash_attn_bwd_workspace_bytes.argtypes = [P]
        L.dash_attn_bwd_attend_prefill_tc.restype = ctypes.c_int
        L.dash_attn_bwd_attend_prefill_tc.argtypes = [P] + [c_void_p] * 11 + [c_size_t, c_void_p]
        L.dash_attn_bwd_select_prefill.restype = ctypes.c_int
        L.dash_attn_bwd_select_prefill.argtypes = [P] + [c_void_p] * 9
        L.dash_attn_bwd_block_summaries.restype = ctypes.c_int
        L.dash_attn_bwd_block_summaries.argtypes = [P, c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]
        L.dash_attn_fwd_prefill.restype = ctypes.c_int
        L.dash_attn_fwd_prefill.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_void_p,
                                            c_void_p, c_void_p, c_size_t, c_void_p]
        L.dash_attn_fwd_decode.restype = ctypes.c_int
        L.dash_attn_fwd_decode.argtypes = [P] + [c_void_p] * 7 + [c_size_t, c_void_p]
        L.dash_attn_block_summaries_paged.restype = ctypes.c_int
        L.dash_attn_block_summaries_paged.argtypes = [P, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_int64,
                                                      c_void_p, c_int32, c_int32, c_void_p, c_void_p]
        L.dash_attn_fwd_decode_paged.restype = ctypes.c_int
        L.dash_attn_fwd_decode_paged.argtypes = [P, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32,
                                                 c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.dash_attn_reset_status.restype = ctypes.c_int
        L.dash_attn_reset_status.argtypes = [c_void_p, c_void_p]
        L.dash_attn_last_status.restype = ctypes.c_int
        L.dash_attn_last_status.argtypes = [c_void_p, c_void_p]
        L.dash_attn_launch_count.restype = c_int64
        L.dash_attn_launch_count.argtypes = []
        L.dash_attn_test_hooks.restype = None
        L.dash_attn_test_hooks.argtypes = [c_int64, c_int32]
        L.dash_attn_strerror.restype = c_char_p
        L.dash_attn_strerror.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


class use_debug_library:
    """Context manager: inside it every binding call goes to libdash_attn_debug.so (built by
    `python -m paper_2605_18753_b200.build --debug`), whose kernels check every index they read from device memory
    and record DASH_ERR_CAPACITY instead of making a bad access.  Raises if that library has not been built."""

    def __enter__(self):
        global _lib, LIB_PATH
        if not os.path.exists(DEBUG_LIB_PATH):
            raise RuntimeError(f"{DEBUG_LIB_PATH} is missing: build it with `python -m paper_2605_18753_b200.build --debug`")
        self._saved = (_lib, LIB_PATH)
        _lib, LIB_PATH = None, DEBUG_LIB_PATH
        lib()
        return self

    def __exit__(self, *exc):
        global _lib, LIB_PATH
        _lib, LIB_PATH = self._saved
        return False


def strerror(code: int) -> str:
    return lib().dash_attn_strerror(int(code)).decode()


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return c_void_p(t)
    return c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, where: str):
    if rc != DASH_OK:
        raise DashError(rc, where)


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return DASH_F32
    if dt == torch.bfloat16:
        return DASH_BF16
    raise ValueError(f"unsupported dtype {dt}")


def _strides3(t: torch.Tensor, decode_q: bool = False):
    """Element strides (batch, token, head) of a [b, n, h, d] tensor, or of a decode query [b, h, d]."""
    if t.stride(-1) != 1:
        raise ValueError("head_dim axis must be contiguous")
    if decode_q:
        return (t.stride(0), 0, t.stride(1))
    return (t.stride(0), t.stride(1), t.stride(2))


def make_params(*, batch, seq_q, seq_kv, h_q, h_kv, head_dim, block, dtype, alpha, gamma=1.0, sigma=10.0,
                causal=1, local_blocks=0, q_stride=None, k_stride=None, v_stride=None, o_stride=None) -> DashParams:
    """Fills a dash_params; strides default to contiguous [b, n, h, d] (decode Q/O: [b, h, d])."""
    p = DashParams()
    p.struct_size = ctypes.sizeof(DashParams)
    p.batch, p.seq_q, p.seq_kv = batch, seq_q, seq_kv
    p.h_q, p.h_kv, p.head_dim, p.block = h_q, h_kv, head_dim, block
    p.dtype = dtype if isinstance(dtype, int) else _dtype_code(dtype)
    p.causal = causal
    p.alpha, p.gamma, p.sigma = alpha, gamma, sigma
    p.local_blocks = local_blocks
    p.q_to_kv = None
    dq = (seq_q * h_q * head_dim, h_q * head_dim, head_dim) if seq_q == seq_kv else (h_q * head_dim, 0, head_dim)
    dk = (seq_kv * h_kv * head_dim, h_kv * head_dim, head_dim)
    for name, val, dflt in (("q_stride", q_stride, dq), ("k_stride", k_stride, dk), ("v_stride", v_stride, dk),
                            ("o_stride", o_stride, dq)):
        setattr(p, name, (c_int64 * 3)(*(val if val is not None else dflt)))
    return p


def params_for_prefill(Q, K, V, O, *, block, alpha, gamma=1.0, sigma=10.0, local_blocks=0, causal=1) -> DashParams:
    b, n, h_q, d = Q.shape
    return make_params(batch=b, seq_q=n, seq_kv=K.shape[1], h_q=h_q, h_kv=K.shape[2], head_dim=d, block=block,
                       dtype=Q.dtype, alpha=alpha, gamma=gamma, sigma=sigma, local_blocks=local_blocks, causal=causal,
                       q_stride=_strides3(Q),
                       k_stride=_strides3(K), v_stride=_strides3(V), o_stride=_strides3(O))


def params_for_decode(Q, Kc, Vc, O, *, block, alpha, gamma=1.0, sigma=10.0, local_blocks=0) -> DashParams:
    b, h_q, d = Q.shape
    return make_params(batch=b, seq_q=1, seq_kv=Kc.shape[1], h_q=h_q, h_kv=Kc.shape[2], head_dim=d, block=block,
                       dtype=Q.dtype, alpha=alpha, gamma=gamma, sigma=sigma, local_blocks=local_blocks,
                       q_stride=_strides3(Q, True),
                       k_stride=_strides3(Kc), v_stride=_strides3(Vc), o_stride=_strides3(O, True))


# ---------------------------------------------------------------- sizes and buffers

def dash_attn_workspace_bytes(p: DashParams) -> int:
    return int(lib().dash_attn_workspace_bytes(ctypes.byref(p)))


def dash_attn_list_capacity(p: DashParams) -> int:
    return int(lib().dash_attn_list_capacity(ctypes.byref(p)))


def dash_attn_list_offset(p: DashParams, b: int, kv_head: int, row: int) -> int:
    return int(lib().dash_attn_list_offset(ctypes.byref(p), b, kv_head, row))


def alloc_workspace(p: DashParams, device="cuda") -> torch.Tensor:
    nbytes = dash_attn_workspace_bytes(p)
    if nbytes == 0:
        raise DashError(-1, "dash_attn_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    dash_attn_reset_status(ws)
    return ws


def alloc_routing(p: DashParams, device="cuda", with_tau=False) -> dict:
    """Buffers for dash_attn_select's outputs."""
    T_a = (p.seq_kv + p.block - 1) // p.block
    W = (T_a + 31) // 32
    T_s = p.seq_kv // p.block
    cap = max(dash_attn_list_capacity(p), 1)
    out = {
        "mask": torch.empty(p.batch, p.h_kv, p.seq_q, W, dtype=torch.int32, device=device),
        "count": torch.empty(p.batch, p.h_kv, p.seq_q, dtype=torch.int32, device=device),
        "blk_idx": torch.empty(cap, dtype=torch.int32, device=device),
        "blk_bias": torch.empty(cap, dtype=torch.float32, device=device),
        "tau": torch.empty(p.batch, p.h_q, p.seq_q, dtype=torch.float32, device=device) if with_tau else None,
    }
    return out


def alloc_kbar(p: DashParams, device="cuda") -> torch.Tensor:
    return torch.empty(p.batch, p.h_kv, max(p.seq_kv // p.block, 0), p.head_dim, dtype=torch.float32, device=device)


# ---------------------------------------------------------------- entry points

def dash_attn_block_summaries(p, K, Kbar, qbar=None, qbar_chunk_stride=0, kv_len=None, first_block=0, num_blocks=-1):
    _check(lib().dash_attn_block_summaries(ctypes.byref(p), _ptr(K), _ptr(qbar), qbar_chunk_stride, _ptr(kv_len),
                                           first_block, num_blocks, _ptr(Kbar), _stream()), "dash_attn_block_summaries")


def dash_attn_select(p, Q, Kbar, mask, count, blk_idx, blk_bias, workspace, tau=None, kv_len=None):
    _check(lib().dash_attn_select(ctypes.byref(p), _ptr(Q), _ptr(Kbar), _ptr(kv_len), _ptr(mask), _ptr(count),
                                  _ptr(blk_idx), _ptr(blk_bias), _ptr(tau), _ptr(workspace), workspace.numel(),
                                  _stream()), "dash_attn_select")


def dash_attn_attend_prefill(p, Q, K, V, mask, blk_bias, O, workspace):
    _check(lib().dash_attn_attend_prefill(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(mask), _ptr(blk_bias),
                                          _ptr(O), _ptr(workspace), workspace.numel(), _stream()),
           "dash_attn_attend_prefill")


def dash_attn_attend_decode(p, Q, Kc, Vc, kv_len, count, blk_idx, blk_bias, O, workspace):
    _check(lib().dash_attn_attend_decode(ctypes.byref(p), _ptr(Q), _ptr(Kc), _ptr(Vc), _ptr(kv_len), _ptr(count),
                                         _ptr(blk_idx), _ptr(blk_bias), _ptr(O), _ptr(workspace), workspace.numel(),
                                         _stream()), "dash_attn_attend_decode")


def dash_attn_attend_decode_static(p, Q, Kc, Vc, kv_len, count, blk_idx, blk_bias, O):
    """Split-KV decode attention for callers that cannot allocate device memory: no workspace argument, the
    split partials use a fixed 4 MiB array inside the library.  Calls must not overlap on the GPU."""
    _check(lib().dash_attn_attend_decode_static(ctypes.byref(p), _ptr(Q), _ptr(Kc), _ptr(Vc), _ptr(kv_len),
                                                _ptr(count), _ptr(blk_idx), _ptr(blk_bias), _ptr(O), _stream()),
           "dash_attn_attend_decode_static")


def dash_attn_bwd_attend_prefill(p, Q, K, V, dO, mask, blk_bias, dQ, dK, dV, dbias):
    """Backward of Stage 2 (prefill) with the routing held fixed; dK / dV fp32 [b, n, h_kv, d], dbias like blk_bias."""
    _check(lib().dash_attn_bwd_attend_prefill(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(mask),
                                              _ptr(blk_bias), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dbias), _stream()),
           "dash_attn_bwd_attend_prefill")


def alloc_bwd_workspace(p: DashParams, device="cuda") -> torch.Tensor:
    nbytes = int(lib().dash_attn_bwd_workspace_bytes(ctypes.byref(p)))
    if nbytes == 0:
        raise DashError(-1, "dash_attn_bwd_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    dash_attn_reset_status(ws)
    return ws


def dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, mask, blk_bias, dQ, dK, dV, dbias, bwd_workspace):
    """The same gradients from the tensor-core kernels (bf16, head_dim 128, chunks of 64 / 128); raises DashError with
    DASH_ERR_UNSUPPORTED for other shapes."""
    _check(lib().dash_attn_bwd_attend_prefill_tc(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(mask),
                                                 _ptr(blk_bias), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dbias),
                                                 _ptr(bwd_workspace), bwd_workspace.numel(), _stream()),
           "dash_attn_bwd_attend_prefill_tc")


def dash_attn_bwd_select_prefill(p, Q, Kbar, count, blk_idx, tau, dbias, dQ_route, dKbar):
    """Backward of Stage 1 (prefill): dbias -> dQ_route (fp32 [b, n, h_q, d]) and dKbar (fp32 like Kbar)."""
    _check(lib().dash_attn_bwd_select_prefill(ctypes.byref(p), _ptr(Q), _ptr(Kbar), _ptr(count), _ptr(blk_idx), _ptr(tau),
                                              _ptr(dbias), _ptr(dQ_route), _ptr(dKbar), _stream()),
           "dash_attn_bwd_select_prefill")


def dash_attn_bwd_block_summaries(p, K, dKbar, dK, qbar=None, qbar_chunk_stride=0, dqbar=None):
    """Backward of Stage 0: adds the summaries' share to dK (fp32 [b, n, h_kv, d]); dqbar gets the summary query's gradient."""
    _check(lib().dash_attn_bwd_block_summaries(ctypes.byref(p), _ptr(K), _ptr(qbar), qbar_chunk_stride, _ptr(dKbar),
                                               _ptr(dK), _ptr(dqbar), _stream()), "dash_attn_bwd_block_summaries")


def dash_attn_fwd_prefill(p, Q, K, V, O, workspace, qbar=None, qbar_chunk_stride=0, Kbar=None, mask_out=None):
    _check(lib().dash_attn_fwd_prefill(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(qbar), qbar_chunk_stride,
                                       _ptr(Kbar), _ptr(O), _ptr(mask_out), _ptr(workspace), workspace.numel(),
                                       _stream()), "dash_attn_fwd_prefill")


def dash_attn_fwd_decode(p, Q, Kc, Vc, Kbar, kv_len, O, workspace):
    _check(lib().dash_attn_fwd_decode(ctypes.byref(p), _ptr(Q), _ptr(Kc), _ptr(Vc), _ptr(Kbar), _ptr(kv_len),
                                      _ptr(O), _ptr(workspace), workspace.numel(), _stream()), "dash_attn_fwd_decode")


def params_for_paged_decode(Q, Kpool, Vpool, O, *, max_pages, block, alpha, gamma=1.0, sigma=10.0, local_blocks=0):
    """Decode parameters over pools [num_pages, page_size, h_kv, d]: seq_kv is the logical capacity max_pages * page_size
    and the K / V strides are those of (page, token in page, head)."""
    b, h_q, d = Q.shape
    return make_params(batch=b, seq_q=1, seq_kv=max_pages * Kpool.shape[1], h_q=h_q, h_kv=Kpool.shape[2], head_dim=d,
                       block=block, dtype=Q.dtype, alpha=alpha, gamma=gamma, sigma=sigma, local_blocks=local_blocks,
                       q_stride=_strides3(Q, True), k_stride=_strides3(Kpool), v_stride=_strides3(Vpool),
                       o_stride=_strides3(O, True))


def dash_attn_block_summaries_paged(p, Kpool, page_table, Kbar, qbar=None, qbar_chunk_stride=0, kv_len=None,
                                    first_block=0, num_blocks=-1):
    _check(lib().dash_attn_block_summaries_paged(ctypes.byref(p), _ptr(Kpool), _ptr(page_table), Kpool.shape[1],
                                                 page_table.shape[1], Kpool.shape[0], _ptr(qbar), qbar_chunk_stride,
                                                 _ptr(kv_len), first_block, num_blocks, _ptr(Kbar), _stream()),
           "dash_attn_block_summaries_paged")


def dash_attn_fwd_decode_paged(p, Q, Kpool, Vpool, page_table, Kbar, kv_len, O, workspace):
    _check(lib().dash_attn_fwd_decode_paged(ctypes.byref(p), _ptr(Q), _ptr(Kpool), _ptr(Vpool), _ptr(page_table),
                                            Kpool.shape[1], page_table.shape[1], Kpool.shape[0], _ptr(Kbar), _ptr(kv_len),
                                            _ptr(O), _ptr(workspace), workspace.numel(), _stream()),
           "dash_attn_fwd_decode_paged")


def dash_attn_reset_status(workspace):
    _check(lib().dash_attn_reset_status(_ptr(workspace), _stream()), "dash_attn_reset_status")


def dash_attn_last_status(workspace) -> int:
    return int(lib().dash_attn_last_status(_ptr(workspace), _stream()))


def dash_attn_test_hooks(wait_limit_cycles: int = 0, skip_own_k_load: int = 0) -> None:
    """Test-suite switches (see the header); calling it without arguments restores the defaults."""
    lib().dash_attn_test_hooks(int(wait_limit_cycles), int(skip_own_k_load))


def dash_attn_launch_count() -> int:
    return int(lib().dash_attn_launch_count())

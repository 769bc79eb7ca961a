"""ctypes binding of ``libseer.so`` (the C ABI declared in ``include/seer.h``).

Argument marshalling only: tensors are passed as raw device pointers plus element strides,
every step of the decode path runs in the library's CUDA kernels.  There is no fallback:
if the shared library is missing or fails to load, importing the symbols raises.

PyTorch is used for device memory and streams; K/V-like tensors are ``[B, Hkv, S, d]``
views (any memory order with unit channel stride), paged caches ``[pages, Hkv, P, d]`` views.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libseer.so")

SEER_OK = 0
SEER_ERR_INVALID_ARG = 1
SEER_ERR_UNSUPPORTED = 2
SEER_ERR_WORKSPACE = 3
SEER_ERR_CUDA = 4
SEER_ERR_BAD_INDEX = 5
SEER_ERR_TIMEOUT = 6

EXPORTS = [
    "seer_create", "seer_destroy", "seer_status_string", "seer_last_error",
    "seer_get_device_status", "seer_workspace_bytes", "seer_launch_count",
    "seer_dense_decode", "seer_sparse_decode", "seer_gate_select", "seer_kcomp_append",
    "seer_gate_select_static", "seer_decode_step", "seer_gate_select_threshold",
    "seer_sparse_decode_multi", "seer_dense_decode_multi", "seer_gate_select_multi", "seer_decode_step_multi",
    "seer_debug_wait_timeout", "seer_gate_select_threshold_multi", "seer_debug_read_bandwidth",
]


class SeerShape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int), ("num_q_heads", ctypes.c_int), ("num_kv_heads", ctypes.c_int),
                ("head_dim", ctypes.c_int), ("block_size", ctypes.c_int), ("sm_scale", ctypes.c_float)]


class SeerKV(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("stride_batch", ctypes.c_int64), ("stride_head", ctypes.c_int64),
                ("stride_token", ctypes.c_int64),
                ("page_table", ctypes.c_void_p), ("page_table_stride", ctypes.c_int64),
                ("page_size", ctypes.c_int), ("num_pages", ctypes.c_int),
                ("seq_lens", ctypes.c_void_p), ("max_seq_len", ctypes.c_int)]


class SeerGate(ctypes.Structure):
    _fields_ = [("d_gate", ctypes.c_int), ("rope_theta", ctypes.c_float),
                ("w_q", ctypes.c_void_p), ("w_k", ctypes.c_void_p), ("kcomp", ctypes.c_void_p),
                ("max_blocks", ctypes.c_int)]


class SeerError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"seer status {status}: {message}")
        self.status = status


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Loads the shared library (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: build it with `python -m paper_2506_08889_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    L.seer_create.restype = i32
    L.seer_create.argtypes = [ctypes.POINTER(vp), i32, ctypes.c_size_t]
    L.seer_destroy.restype = None
    L.seer_destroy.argtypes = [vp]
    L.seer_status_string.restype = ctypes.c_char_p
    L.seer_status_string.argtypes = [i32]
    L.seer_last_error.restype = ctypes.c_char_p
    L.seer_last_error.argtypes = [vp]
    L.seer_get_device_status.restype = i32
    L.seer_get_device_status.argtypes = [vp, vp]
    L.seer_workspace_bytes.restype = ctypes.c_size_t
    L.seer_workspace_bytes.argtypes = [ctypes.POINTER(SeerShape), i32, i32]
    L.seer_launch_count.restype = ctypes.c_uint64
    L.seer_launch_count.argtypes = [vp]
    L.seer_dense_decode.restype = i32
    L.seer_dense_decode.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerKV), vp, vp, vp, vp]
    L.seer_sparse_decode.restype = i32
    L.seer_sparse_decode.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerKV), vp, vp, vp, i32,
                                     vp, vp, vp]
    L.seer_sparse_decode_multi.restype = i32
    L.seer_sparse_decode_multi.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerKV), vp, i32, vp, vp,
                                           i32, vp, vp, vp]
    L.seer_dense_decode_multi.restype = i32
    L.seer_dense_decode_multi.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerKV), vp, i32, vp, vp, vp]
    L.seer_gate_select_multi.restype = i32
    L.seer_gate_select_multi.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerGate), vp, vp, vp, i32, i32,
                                         vp, vp, i32, vp, vp]
    L.seer_gate_select.restype = i32
    L.seer_gate_select.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerGate), vp, vp, vp, i32,
                                   vp, vp, i32, vp, vp]
    L.seer_kcomp_append.restype = i32
    L.seer_kcomp_append.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerGate), vp, vp,
                                    i64, i64, i64, i32, i32, i32, vp]
    L.seer_gate_select_threshold.restype = i32
    L.seer_gate_select_threshold.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerGate), vp, vp, vp,
                                             ctypes.c_float, vp, vp, i32, vp, vp]
    L.seer_gate_select_threshold_multi.restype = i32
    L.seer_gate_select_threshold_multi.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerGate), vp, vp, vp, i32,
                                                   ctypes.c_float, vp, vp, i32, vp, vp]
    L.seer_decode_step_multi.restype = i32
    L.seer_decode_step_multi.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerKV), ctypes.POINTER(SeerGate),
                                         vp, vp, i32, vp, i64, i64, i64, i32, i32, vp, vp, i32, vp, vp, vp]
    L.seer_decode_step.restype = i32
    L.seer_decode_step.argtypes = [vp, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerKV), ctypes.POINTER(SeerGate),
                                   vp, vp, vp, i64, i64, i64, i32, i32, vp, vp, i32, vp, vp, vp]
    L.seer_debug_wait_timeout.restype = i32
    L.seer_debug_wait_timeout.argtypes = [vp, i32, vp]
    L.seer_debug_read_bandwidth.restype = i32
    L.seer_debug_read_bandwidth.argtypes = [vp, vp, ctypes.c_size_t, vp, vp]
    L.seer_gate_select_static.restype = i32
    L.seer_gate_select_static.argtypes = [i32, ctypes.POINTER(SeerShape), ctypes.POINTER(SeerGate), vp, vp, i32,
                                          vp, vp, i32, vp, vp, ctypes.c_char_p, ctypes.c_size_t]
    _lib = L
    return L


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def make_shape(batch, num_q_heads, num_kv_heads, head_dim, block_size, sm_scale) -> SeerShape:
    return SeerShape(batch, num_q_heads, num_kv_heads, head_dim, block_size, sm_scale)


def make_kv(k: torch.Tensor, v: torch.Tensor, seq_lens: torch.Tensor, max_seq_len: Optional[int] = None,
            page_table: Optional[torch.Tensor] = None, page_size: int = 0) -> SeerKV:
    """k, v: [B, Hkv, S, d] views (contiguous layout) or [pages, Hkv, P, d] views (paged)."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16
    assert k.shape == v.shape and k.stride() == v.stride() and k.stride(3) == 1
    assert seq_lens.dtype == torch.int32 and seq_lens.is_contiguous()
    kv = SeerKV()
    kv.k, kv.v = k.data_ptr(), v.data_ptr()
    kv.stride_batch, kv.stride_head, kv.stride_token = k.stride(0), k.stride(1), k.stride(2)
    kv.seq_lens = seq_lens.data_ptr()
    if page_table is None:
        kv.page_table, kv.page_table_stride, kv.page_size, kv.num_pages = None, 0, 0, 0
        kv.max_seq_len = int(max_seq_len if max_seq_len is not None else k.shape[2])
    else:
        assert page_table.dtype == torch.int32 and page_table.dim() == 2 and page_table.stride(1) == 1
        kv.page_table = page_table.data_ptr()
        kv.page_table_stride = page_table.stride(0)
        kv.page_size = int(page_size or k.shape[2])
        kv.num_pages = int(k.shape[0])
        kv.max_seq_len = int(max_seq_len if max_seq_len is not None else page_table.shape[1] * kv.page_size)
    return kv


def make_gate(d_gate: int, rope_theta: float, w_q: Optional[torch.Tensor], w_k: Optional[torch.Tensor],
              kcomp: Optional[torch.Tensor], max_blocks: int) -> SeerGate:
    g = SeerGate()
    g.d_gate, g.rope_theta, g.max_blocks = int(d_gate), float(rope_theta), int(max_blocks)
    g.w_q = None if w_q is None else w_q.data_ptr()
    g.w_k = None if w_k is None else w_k.data_ptr()
    g.kcomp = None if kcomp is None else kcomp.data_ptr()
    return g


class Context:
    """Owns one ``seer_ctx`` (device workspace).  One context per concurrent stream."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self._h = ctypes.c_void_p()
        st = lib().seer_create(ctypes.byref(self._h), int(device), int(workspace_bytes))
        if st != SEER_OK:
            raise SeerError(st, lib().seer_status_string(st).decode() + " (seer_create)")
        self.device = int(device)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().seer_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != SEER_OK:
            raise SeerError(st, lib().seer_last_error(self._h).decode())

    def launch_count(self) -> int:
        return int(lib().seer_launch_count(self._h))

    def device_status(self, stream=None) -> int:
        return int(lib().seer_get_device_status(self._h, _stream(stream)))

    def seer_debug_wait_timeout(self, polls: int, stream=None):
        self._check(lib().seer_debug_wait_timeout(self._h, int(polls), _stream(stream)))

    def seer_debug_read_bandwidth(self, src, nbytes: int, checksum, stream=None):
        self._check(lib().seer_debug_read_bandwidth(self._h, _ptr(src), ctypes.c_size_t(int(nbytes)), _ptr(checksum),
                                                    _stream(stream)))

    # ---- the four operations (names follow the C ABI) ------------------------------------
    def seer_dense_decode(self, shape: SeerShape, kv: SeerKV, q, out, lse=None, stream=None):
        self._check(lib().seer_dense_decode(self._h, ctypes.byref(shape), ctypes.byref(kv), _ptr(q), _ptr(out),
                                            _ptr(lse), _stream(stream)))

    def seer_sparse_decode(self, shape: SeerShape, kv: SeerKV, q, block_idx, block_cnt, max_sel, out, lse=None,
                           stream=None):
        self._check(lib().seer_sparse_decode(self._h, ctypes.byref(shape), ctypes.byref(kv), _ptr(q),
                                             _ptr(block_idx), _ptr(block_cnt), int(max_sel), _ptr(out),
                                             _ptr(lse), _stream(stream)))

    def seer_sparse_decode_multi(self, shape: SeerShape, kv: SeerKV, q, q_len, block_idx, block_cnt, max_sel, out,
                                 lse=None, stream=None):
        self._check(lib().seer_sparse_decode_multi(self._h, ctypes.byref(shape), ctypes.byref(kv), _ptr(q),
                                                   int(q_len), _ptr(block_idx), _ptr(block_cnt), int(max_sel),
                                                   _ptr(out), _ptr(lse), _stream(stream)))

    def seer_dense_decode_multi(self, shape: SeerShape, kv: SeerKV, q, q_len, out, lse=None, stream=None):
        self._check(lib().seer_dense_decode_multi(self._h, ctypes.byref(shape), ctypes.byref(kv), _ptr(q),
                                                  int(q_len), _ptr(out), _ptr(lse), _stream(stream)))

    def seer_gate_select(self, shape: SeerShape, gate: SeerGate, seq_lens, q_nope, scores_in, token_budget,
                         block_idx, block_cnt, max_sel, scores_out=None, stream=None):
        self._check(lib().seer_gate_select(self._h, ctypes.byref(shape), ctypes.byref(gate), _ptr(seq_lens),
                                           _ptr(q_nope), _ptr(scores_in), int(token_budget), _ptr(block_idx),
                                           _ptr(block_cnt), int(max_sel), _ptr(scores_out), _stream(stream)))

    def seer_gate_select_multi(self, shape: SeerShape, gate: SeerGate, seq_lens, q_nope, scores_in, q_len,
                               token_budget, block_idx, block_cnt, max_sel, scores_out=None, stream=None):
        self._check(lib().seer_gate_select_multi(self._h, ctypes.byref(shape), ctypes.byref(gate), _ptr(seq_lens),
                                                 _ptr(q_nope), _ptr(scores_in), int(q_len), int(token_budget),
                                                 _ptr(block_idx), _ptr(block_cnt), int(max_sel), _ptr(scores_out),
                                                 _stream(stream)))

    def seer_gate_select_threshold(self, shape: SeerShape, gate: SeerGate, seq_lens, q_nope, scores_in, threshold,
                                   block_idx, block_cnt, max_sel, scores_out=None, stream=None):
        self._check(lib().seer_gate_select_threshold(self._h, ctypes.byref(shape), ctypes.byref(gate),
                                                     _ptr(seq_lens), _ptr(q_nope), _ptr(scores_in),
                                                     ctypes.c_float(threshold), _ptr(block_idx), _ptr(block_cnt),
                                                     int(max_sel), _ptr(scores_out), _stream(stream)))

    def seer_gate_select_threshold_multi(self, shape: SeerShape, gate: SeerGate, seq_lens, q_nope, scores_in, q_len,
                                         threshold, block_idx, block_cnt, max_sel, scores_out=None, stream=None):
        self._check(lib().seer_gate_select_threshold_multi(self._h, ctypes.byref(shape), ctypes.byref(gate),
                                                           _ptr(seq_lens), _ptr(q_nope), _ptr(scores_in), int(q_len),
                                                           ctypes.c_float(threshold), _ptr(block_idx), _ptr(block_cnt),
                                                           int(max_sel), _ptr(scores_out), _stream(stream)))

    def seer_kcomp_append(self, shape: SeerShape, gate: SeerGate, seq_lens, k_nope, rows_block_local=False,
                          first_block=-1, num_blocks=1, stream=None):
        """k_nope: [B, Hkv, rows, d] view with unit channel stride."""
        assert k_nope.dtype == torch.bfloat16 and k_nope.stride(3) == 1
        self._check(lib().seer_kcomp_append(self._h, ctypes.byref(shape), ctypes.byref(gate), _ptr(seq_lens),
                                            _ptr(k_nope), k_nope.stride(0), k_nope.stride(1), k_nope.stride(2),
                                            int(bool(rows_block_local)), int(first_block), int(num_blocks),
                                            _stream(stream)))

    def seer_decode_step(self, shape: SeerShape, kv: SeerKV, gate: SeerGate, q, q_nope, k_nope, token_budget,
                         block_idx, block_cnt, max_sel, out, lse=None, rows_block_local=False, stream=None):
        """Compressed-K append (skipped if k_nope is None) + gate selection + sparse decode in one call."""
        sb = sh = st = 0
        if k_nope is not None:
            assert k_nope.dtype == torch.bfloat16 and k_nope.stride(3) == 1
            sb, sh, st = k_nope.stride(0), k_nope.stride(1), k_nope.stride(2)
        self._check(lib().seer_decode_step(self._h, ctypes.byref(shape), ctypes.byref(kv), ctypes.byref(gate),
                                           _ptr(q), _ptr(q_nope), _ptr(k_nope), sb, sh, st,
                                           int(bool(rows_block_local)), int(token_budget), _ptr(block_idx),
                                           _ptr(block_cnt), int(max_sel), _ptr(out), _ptr(lse), _stream(stream)))


    def seer_decode_step_multi(self, shape: SeerShape, kv: SeerKV, gate: SeerGate, q, q_nope, q_len, k_nope,
                               token_budget, block_idx, block_cnt, max_sel, out, lse=None, rows_block_local=False,
                               stream=None):
        """The step for q_len query tokens per sequence (q, q_nope, out: [B,q_len,Hq,d])."""
        sb = sh = st = 0
        if k_nope is not None:
            assert k_nope.dtype == torch.bfloat16 and k_nope.stride(3) == 1
            sb, sh, st = k_nope.stride(0), k_nope.stride(1), k_nope.stride(2)
        self._check(lib().seer_decode_step_multi(self._h, ctypes.byref(shape), ctypes.byref(kv), ctypes.byref(gate),
                                                 _ptr(q), _ptr(q_nope), int(q_len), _ptr(k_nope), sb, sh, st,
                                                 int(bool(rows_block_local)), int(token_budget), _ptr(block_idx),
                                                 _ptr(block_cnt), int(max_sel), _ptr(out), _ptr(lse),
                                                 _stream(stream)))


STATIC_SCRATCH_BYTES = 1 << 20


def seer_gate_select_static(device: int, shape: SeerShape, gate: SeerGate, seq_lens, q_nope, token_budget,
                            block_idx, block_cnt, max_sel, scores_out=None, stream=None):
    """Gate scoring + selection for callers that may not allocate device memory: no context, the
    scratch lives in a fixed array inside the library (see ``seer_gate_select_static`` in seer.h)."""
    buf = ctypes.create_string_buffer(256)
    st = lib().seer_gate_select_static(int(device), ctypes.byref(shape), ctypes.byref(gate), _ptr(seq_lens),
                                       _ptr(q_nope), int(token_budget), _ptr(block_idx), _ptr(block_cnt),
                                       int(max_sel), _ptr(scores_out), _stream(stream), buf, len(buf))
    if st != SEER_OK:
        raise SeerError(st, buf.value.decode())

"""ctypes front end of the fp64 CPU oracle (``seer_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, by the smoke check and by
the benchmark's CPU-baseline leg.  Nothing in the product package imports it, and
it imports nothing from the product package.

bf16 tensors cross this interface as ``numpy.uint16`` arrays holding the raw bit
patterns; K/V-like arrays are ``[B, Hkv, S, d]`` views whose element strides are
passed through, so any layout with unit channel stride works.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "seer_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP for the outer loops only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_round_bf16.restype = ctypes.c_uint16
        _lib.oracle_round_bf16.argtypes = [ctypes.c_double]
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(ctypes.c_int(n))


def round_bf16(x: float) -> int:
    return int(lib().oracle_round_bf16(float(x)))


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a, name):
    a = np.asarray(a)
    if a.dtype != np.uint16:
        raise TypeError(f"{name}: expected raw bf16 bits as uint16, got {a.dtype}")
    return a


def _kv_strides(k, v=None):
    if k.ndim != 4 or k.strides[3] != k.itemsize:
        raise ValueError("K/V must be [B,Hkv,S,d] views with unit channel stride")
    if v is not None and (v.strides != k.strides or v.shape != k.shape):
        raise ValueError("K and V must share shape and strides")
    return tuple(ctypes.c_int64(s // k.itemsize) for s in k.strides[:3])


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def dense(q, k, v, seq_lens, scale):
    """Dense decode attention.  Returns (out [B,Hq,d] f64, lse [B,Hq] f64)."""
    q = np.ascontiguousarray(_u16(q, "q")); k = _u16(k, "k"); v = _u16(v, "v")
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    sb, sh, st = _kv_strides(k, v)
    seq_lens = _i32(seq_lens)
    out = np.zeros((B, Hq, d), np.float64)
    lse = np.zeros((B, Hq), np.float64)
    lib().oracle_dense(_p(q), _p(k), _p(v), sb, sh, st, _p(seq_lens),
                       ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d),
                       ctypes.c_double(scale), _p(out), _p(lse))
    return out, lse


def sparse(q, k, v, seq_lens, block_idx, block_cnt, block_size, scale):
    """Block-sparse decode attention over the listed blocks."""
    q = np.ascontiguousarray(_u16(q, "q")); k = _u16(k, "k"); v = _u16(v, "v")
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    sb, sh, st = _kv_strides(k, v)
    seq_lens = _i32(seq_lens)
    block_idx = _i32(block_idx)
    assert block_idx.shape[:2] == (B, Hkv)
    max_sel = block_idx.shape[2]
    cnt = None if block_cnt is None else _i32(block_cnt)
    out = np.zeros((B, Hq, d), np.float64)
    lse = np.zeros((B, Hq), np.float64)
    lib().oracle_sparse(_p(q), _p(k), _p(v), sb, sh, st, _p(seq_lens), _p(block_idx), _p(cnt),
                        ctypes.c_int(max_sel), ctypes.c_int(B), ctypes.c_int(Hq),
                        ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_int(block_size),
                        ctypes.c_double(scale), _p(out), _p(lse))
    return out, lse


def sparse_multi(q, k, v, seq_lens, block_idx, block_cnt, block_size, scale):
    """Block-sparse attention for T query tokens per sequence (the last T cached tokens), causal
    among them, one block list per (sequence, KV head).  q: [B,T,Hq,d] bf16 bits.
    Returns (out [B,T,Hq,d] f64, lse [B,T,Hq] f64)."""
    q = np.ascontiguousarray(_u16(q, "q")); k = _u16(k, "k"); v = _u16(v, "v")
    B, T, Hq, d = q.shape
    Hkv = k.shape[1]
    sb, sh, st = _kv_strides(k, v)
    seq_lens = _i32(seq_lens)
    block_idx = _i32(block_idx)
    assert block_idx.shape[:2] == (B, Hkv)
    max_sel = block_idx.shape[2]
    cnt = None if block_cnt is None else _i32(block_cnt)
    out = np.zeros((B, T, Hq, d), np.float64)
    lse = np.zeros((B, T, Hq), np.float64)
    lib().oracle_sparse_multi(_p(q), _p(k), _p(v), sb, sh, st, _p(seq_lens), _p(block_idx), _p(cnt),
                              ctypes.c_int(max_sel), ctypes.c_int(B), ctypes.c_int(T), ctypes.c_int(Hq),
                              ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_int(block_size),
                              ctypes.c_double(scale), _p(out), _p(lse))
    return out, lse


def kcomp(k_nope, w_k, block_size, first_block, num_blocks, max_blocks, theta,
          kc_bf16=None):
    """K-branch entries for blocks first_block..first_block+num_blocks-1.

    Returns (kc_bf16 [B,Hkv,max_blocks,dg] uint16, kc_f64 same shape); entries
    outside the range keep the values of the ``kc_bf16`` passed in (zeros if None).
    """
    k_nope = _u16(k_nope, "k_nope")
    w_k = np.ascontiguousarray(_u16(w_k, "w_k"))
    B, Hkv, _, d = k_nope.shape
    dg = w_k.shape[1]
    assert w_k.shape == (Hkv, dg, 3 * d)
    sb, sh, st = _kv_strides(k_nope)
    if kc_bf16 is None:
        kc_bf16 = np.zeros((B, Hkv, max_blocks, dg), np.uint16)
    else:
        kc_bf16 = np.ascontiguousarray(_u16(kc_bf16, "kc")).copy()
    kc_f64 = np.zeros((B, Hkv, max_blocks, dg), np.float64)
    lib().oracle_kcomp(_p(k_nope), sb, sh, st, _p(w_k), ctypes.c_int(B), ctypes.c_int(Hkv),
                       ctypes.c_int(d), ctypes.c_int(dg), ctypes.c_int(block_size),
                       ctypes.c_int(first_block), ctypes.c_int(num_blocks),
                       ctypes.c_int(max_blocks), ctypes.c_double(theta), _p(kc_bf16), _p(kc_f64))
    return kc_bf16, kc_f64


def scores(q_nope, w_q, kc, n_entries, qpos, theta):
    """Gate scores.  Returns (scores [B,Hkv,max_blocks] f64, q_gate [B,Hkv,dg] f64)."""
    q_nope = np.ascontiguousarray(_u16(q_nope, "q_nope"))
    w_q = np.ascontiguousarray(_u16(w_q, "w_q"))
    kc = np.ascontiguousarray(_u16(kc, "kc"))
    B, Hq, d = q_nope.shape
    _, Hkv, max_blocks, dg = kc.shape
    assert w_q.shape == (Hkv, dg, (Hq // Hkv) * d)
    n_entries = _i32(n_entries); qpos = _i32(qpos)
    sc = np.zeros((B, Hkv, max_blocks), np.float64)
    qg = np.zeros((B, Hkv, dg), np.float64)
    lib().oracle_scores(_p(q_nope), _p(w_q), _p(kc), _p(n_entries), _p(qpos),
                        ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d),
                        ctypes.c_int(dg), ctypes.c_int(max_blocks), ctypes.c_double(theta),
                        _p(sc), _p(qg))
    return sc, qg


def select(scores_f32, seq_lens, block_size, token_budget, max_sel):
    """Token-budget top-k with the forced last block.  Returns (idx, cnt) int32."""
    s = np.ascontiguousarray(np.asarray(scores_f32))
    if s.dtype != np.float32:
        raise TypeError("selection is defined on fp32 scores")
    B, Hkv, max_blocks = s.shape
    seq_lens = _i32(seq_lens)
    idx = np.zeros((B, Hkv, max_sel), np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    lib().oracle_select(_p(s), _p(seq_lens), ctypes.c_int(B), ctypes.c_int(Hkv),
                        ctypes.c_int(block_size), ctypes.c_int(max_blocks),
                        ctypes.c_int(token_budget), ctypes.c_int(max_sel), _p(idx), _p(cnt))
    return idx, cnt


def scores_multi(q_nope, w_q, kc, seq_lens, block_size, theta):
    """Gate scores for T query tokens per sequence: per block the largest of the tokens' scores, over
    the blocks wholly before the first query token.  q_nope: [B,T,Hq,d].  Returns [B,Hkv,max_blocks] f64."""
    q_nope = np.ascontiguousarray(_u16(q_nope, "q_nope"))
    w_q = np.ascontiguousarray(_u16(w_q, "w_q"))
    kc = np.ascontiguousarray(_u16(kc, "kc"))
    B, T, Hq, d = q_nope.shape
    _, Hkv, max_blocks, dg = kc.shape
    assert w_q.shape == (Hkv, dg, (Hq // Hkv) * d)
    seq_lens = _i32(seq_lens)
    sc = np.zeros((B, Hkv, max_blocks), np.float64)
    lib().oracle_scores_multi(_p(q_nope), _p(w_q), _p(kc), _p(seq_lens), ctypes.c_int(T),
                              ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d),
                              ctypes.c_int(dg), ctypes.c_int(max_blocks), ctypes.c_int(block_size),
                              ctypes.c_double(theta), _p(sc))
    return sc


def select_multi(scores_f32, seq_lens, block_size, token_budget, q_len, max_sel):
    """Token-budget top-k for q_len query tokens: the blocks holding the query tokens are forced."""
    s = np.ascontiguousarray(np.asarray(scores_f32))
    if s.dtype != np.float32:
        raise TypeError("selection is defined on fp32 scores")
    B, Hkv, max_blocks = s.shape
    seq_lens = _i32(seq_lens)
    idx = np.zeros((B, Hkv, max_sel), np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    lib().oracle_select_multi(_p(s), _p(seq_lens), ctypes.c_int(B), ctypes.c_int(Hkv),
                              ctypes.c_int(block_size), ctypes.c_int(max_blocks),
                              ctypes.c_int(token_budget), ctypes.c_int(q_len), ctypes.c_int(max_sel),
                              _p(idx), _p(cnt))
    return idx, cnt


def select_threshold(scores_f32, seq_lens, block_size, tau, max_sel):
    """Threshold selection on softmax(scores) with the forced last block.
    Returns (idx, cnt, probs f64 [B,Hkv,max_blocks])."""
    s = np.ascontiguousarray(np.asarray(scores_f32))
    if s.dtype != np.float32:
        raise TypeError("selection is defined on fp32 scores")
    B, Hkv, max_blocks = s.shape
    seq_lens = _i32(seq_lens)
    idx = np.zeros((B, Hkv, max_sel), np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    probs = np.zeros((B, Hkv, max_blocks), np.float64)
    lib().oracle_select_threshold(_p(s), _p(seq_lens), ctypes.c_int(B), ctypes.c_int(Hkv),
                                  ctypes.c_int(block_size), ctypes.c_int(max_blocks), ctypes.c_double(tau),
                                  ctypes.c_int(max_sel), _p(idx), _p(cnt), _p(probs))
    return idx, cnt, probs


def select_threshold_multi(scores_f32, seq_lens, block_size, tau, q_len, max_sel):
    """Threshold selection for q_len query tokens: softmax over the blocks wholly before the first query
    token, the blocks holding the query tokens forced.  Returns (idx, cnt, probs f64 [B,Hkv,max_blocks])."""
    s = np.ascontiguousarray(np.asarray(scores_f32))
    if s.dtype != np.float32:
        raise TypeError("selection is defined on fp32 scores")
    B, Hkv, max_blocks = s.shape
    seq_lens = _i32(seq_lens)
    idx = np.zeros((B, Hkv, max_sel), np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    probs = np.zeros((B, Hkv, max_blocks), np.float64)
    lib().oracle_select_threshold_multi(_p(s), _p(seq_lens), ctypes.c_int(B), ctypes.c_int(Hkv),
                                        ctypes.c_int(block_size), ctypes.c_int(max_blocks), ctypes.c_double(tau),
                                        ctypes.c_int(q_len), ctypes.c_int(max_sel), _p(idx), _p(cnt), _p(probs))
    return idx, cnt, probs


def rope(y, pos, theta):
    """Rotate one fp64 vector (length d_gate) to position ``pos``."""
    y = np.array(y, dtype=np.float64).copy()
    lib().oracle_rope(_p(y), ctypes.c_int(y.shape[0]), ctypes.c_double(pos), ctypes.c_double(theta))
    return y

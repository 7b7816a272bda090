"""ctypes access to the C++ CPU oracle (oracle/falcon_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this.
Arguments are numpy arrays; bf16 tensors travel as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build_oracle import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _lib.oracle_max_threads.restype = C.c_int
    return _lib


def _p(a, ctype):
    return None if a is None else a.ctypes.data_as(C.POINTER(ctype))


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def tree_validate(parent) -> int:
    parent = _i32(parent)
    return int(lib().oracle_tree_validate(_p(parent, C.c_int32), C.c_int32(len(parent))))


def ancestors(parent, i: int):
    parent = _i32(parent)
    out = np.empty(len(parent) + 1, dtype=np.int32)
    n = lib().oracle_ancestors(_p(parent, C.c_int32), C.c_int32(len(parent)), C.c_int32(i), _p(out, C.c_int32))
    if n < 0:
        raise ValueError("malformed tree")
    return out[:n].copy()


def tree_attn(node_off, parent, prefix_len, Hq, Hkv, D, sm_scale, q, k_cache, v_cache, strides,
              k_tree=None, v_tree=None, tree_mask=None, n_threads=0):
    """fp32 [N, Hq, D] attention output.  strides = (b, h, s) in elements."""
    node_off, parent, prefix_len = _i32(node_off), _i32(parent), _i32(prefix_len)
    N = int(node_off[-1])
    out = np.empty((N, Hq, D), dtype=np.float32)
    assert q.dtype == np.uint16 and k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16
    if tree_mask is not None:
        tree_mask = np.ascontiguousarray(tree_mask, dtype=np.uint64)
        assert tree_mask.shape == (N, 2)
    rc = lib().oracle_tree_attn(
        C.c_int32(len(prefix_len)), _p(node_off, C.c_int32), _p(parent, C.c_int32), _p(prefix_len, C.c_int32),
        C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(D), C.c_float(sm_scale), _p(q, C.c_uint16),
        _p(k_cache, C.c_uint16), _p(v_cache, C.c_uint16), C.c_int64(strides[0]), C.c_int64(strides[1]),
        C.c_int64(strides[2]), _p(k_tree, C.c_uint16), _p(v_tree, C.c_uint16), _p(tree_mask, C.c_uint64),
        _p(out, C.c_float), C.c_int(n_threads))
    if rc:
        raise ValueError("oracle_tree_attn failed: %d" % rc)
    return out


def causal_attn(L, T, Hq, Hkv, D, sm_scale, q, k, v):
    out = np.empty((T, Hq, D), dtype=np.float32)
    q, k, v = (np.ascontiguousarray(a, dtype=np.uint16) for a in (q, k, v))
    assert k.shape == (Hkv, L + T, D) and v.shape == k.shape and q.shape == (T, Hq, D)
    rc = lib().oracle_causal_attn(C.c_int32(L), C.c_int32(T), C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(D),
                                  C.c_float(sm_scale), _p(q, C.c_uint16), _p(k, C.c_uint16), _p(v, C.c_uint16),
                                  _p(out, C.c_float))
    if rc:
        raise ValueError("oracle_causal_attn failed: %d" % rc)
    return out


def argmax(logits, vocab=None, n_threads=0):
    """logits: C-contiguous fp32 [N, stride]; the first `vocab` columns of each row are scanned."""
    assert logits.dtype == np.float32 and logits.ndim == 2 and logits.flags.c_contiguous
    N, stride = logits.shape
    V = stride if vocab is None else vocab
    g = np.empty(N, dtype=np.int32)
    rc = lib().oracle_argmax(_p(logits, C.c_float), C.c_int32(N), C.c_int32(V), C.c_int64(stride),
                             _p(g, C.c_int32), C.c_int(n_threads))
    if rc:
        raise ValueError("oracle_argmax failed: %d" % rc)
    return g


def sample_tokens(logits, temperature, u, vocab=None, want_cdf=False, n_threads=0):
    """logits: C-contiguous fp32 [N, stride]; u: fp32 [N] uniforms in [0, 1).  Returns g [N] int32 (and the
    normalised partial sums [N, V] float64 with want_cdf)."""
    assert logits.dtype == np.float32 and logits.ndim == 2 and logits.flags.c_contiguous
    N, stride = logits.shape
    V = stride if vocab is None else vocab
    u = np.ascontiguousarray(u, dtype=np.float32)
    assert u.shape == (N,)
    g = np.empty(N, dtype=np.int32)
    cdf = np.empty((N, V), dtype=np.float64) if want_cdf else None
    rc = lib().oracle_sample_tokens(_p(logits, C.c_float), C.c_int32(N), C.c_int32(V), C.c_int64(stride),
                                    C.c_double(temperature), _p(u, C.c_float), _p(g, C.c_int32),
                                    _p(cdf, C.c_double) if want_cdf else None, C.c_int(n_threads))
    if rc:
        raise ValueError("oracle_sample_tokens failed: %d" % rc)
    return (g, cdf) if want_cdf else g


def lm_head_argmax(feat_bits, head_bits, hidden=None, want_logits=False, n_threads=0):
    """feat_bits: uint16 (bf16 bit patterns) [N, feat_stride]; head_bits: uint16 [V, head_stride]; the first
    `hidden` columns of both are used.  Returns (g [N] int32, best [N] float64[, logits [N, V] float64])."""
    for a in (feat_bits, head_bits):
        assert a.dtype == np.uint16 and a.ndim == 2 and a.flags.c_contiguous
    N, fs = feat_bits.shape
    V, hs = head_bits.shape
    H = min(fs, hs) if hidden is None else hidden
    g = np.empty(N, dtype=np.int32)
    best = np.empty(N, dtype=np.float64)
    logits = np.empty((N, V), dtype=np.float64) if want_logits else None
    rc = lib().oracle_lm_head_argmax(_p(feat_bits, C.c_uint16), C.c_int64(fs), _p(head_bits, C.c_uint16), C.c_int64(hs),
                                     C.c_int32(N), C.c_int32(H), C.c_int32(V), _p(g, C.c_int32), _p(best, C.c_double),
                                     _p(logits, C.c_double) if want_logits else None, C.c_int(n_threads))
    if rc:
        raise ValueError("oracle_lm_head_argmax failed: %d" % rc)
    return (g, best, logits) if want_logits else (g, best)


def topm(logits, m, vocab=None, n_threads=0):
    """logits: C-contiguous fp32 [N, stride].  Returns (values [N, m] fp32, indices [N, m] int32), best first."""
    assert logits.dtype == np.float32 and logits.ndim == 2 and logits.flags.c_contiguous
    N, stride = logits.shape
    V = stride if vocab is None else vocab
    val = np.empty((N, m), dtype=np.float32)
    idx = np.empty((N, m), dtype=np.int32)
    rc = lib().oracle_topm(_p(logits, C.c_float), C.c_int32(N), C.c_int32(V), C.c_int64(stride), C.c_int32(m),
                           _p(val, C.c_float), _p(idx, C.c_int32), C.c_int(n_threads))
    if rc:
        raise ValueError("oracle_topm failed: %d" % rc)
    return val, idx


def _accept(fn, node_off, parent, token, g, path_stride):
    node_off, parent, token, g = _i32(node_off), _i32(parent), _i32(token), _i32(g)
    B = len(node_off) - 1
    path = np.empty((B, path_stride), dtype=np.int32)
    n_path = np.empty(B, dtype=np.int32)
    nxt = np.empty(B, dtype=np.int32)
    rc = fn(C.c_int32(B), _p(node_off, C.c_int32), _p(parent, C.c_int32), _p(token, C.c_int32), _p(g, C.c_int32),
            _p(path, C.c_int32), C.c_int32(path_stride), _p(n_path, C.c_int32), _p(nxt, C.c_int32))
    if rc:
        raise ValueError("oracle accept failed: %d" % rc)
    return path, n_path, nxt


def tree_accept(node_off, parent, token, g, path_stride=128):
    return _accept(lib().oracle_tree_accept, node_off, parent, token, g, path_stride)


def bruteforce_accept(node_off, parent, token, g, path_stride=128):
    return _accept(lib().oracle_bruteforce_accept, node_off, parent, token, g, path_stride)


def kv_compact(node_off, prefix_len, Hkv, D, cache, strides, s_cap, path, n_path, tree_rows=None):
    """Compacts `cache` (uint16 numpy array, modified in place); returns new_len."""
    node_off, prefix_len, n_path = _i32(node_off), _i32(prefix_len), _i32(n_path)
    path = np.ascontiguousarray(path, dtype=np.int32)
    assert cache.dtype == np.uint16 and cache.flags.c_contiguous
    new_len = np.empty(len(prefix_len), dtype=np.int32)
    rc = lib().oracle_kv_compact(
        C.c_int32(len(prefix_len)), _p(node_off, C.c_int32), _p(prefix_len, C.c_int32), C.c_int32(Hkv),
        C.c_int32(D), _p(cache, C.c_uint16), C.c_int64(strides[0]), C.c_int64(strides[1]), C.c_int64(strides[2]),
        C.c_int32(s_cap), _p(tree_rows, C.c_uint16), _p(path, C.c_int32), C.c_int32(path.shape[1]),
        _p(n_path, C.c_int32), _p(new_len, C.c_int32))
    if rc:
        raise ValueError("oracle_kv_compact failed: %d" % rc)
    return new_len


def feature_gather(node_off, path, n_path, token, feat, out_rows=None, hidden=None, fill=0):
    """Accepted tokens and features along the path: feat uint16 [N, row stride >= hidden] -> (feat_out uint16
    [B, out_rows, hidden], tok_out int32 [B, out_rows]); rows past n_path[b] keep `fill`.  `hidden` defaults
    to the row length of `feat`."""
    node_off, n_path, token = _i32(node_off), _i32(n_path), _i32(token)
    path = np.ascontiguousarray(path, dtype=np.int32)
    feat = np.ascontiguousarray(feat)
    assert feat.dtype == np.uint16 and feat.ndim == 2
    B = len(n_path)
    hidden = feat.shape[1] if hidden is None else hidden
    stride = feat.shape[1]
    out_rows = path.shape[1] if out_rows is None else out_rows
    feat_out = np.full((B, out_rows, hidden), fill, dtype=np.uint16)
    tok_out = np.full((B, out_rows), fill, dtype=np.int32)
    rc = lib().oracle_feature_gather(
        C.c_int32(B), _p(node_off, C.c_int32), _p(path, C.c_int32), C.c_int32(path.shape[1]), _p(n_path, C.c_int32),
        _p(token, C.c_int32), _p(feat, C.c_uint16), C.c_int32(hidden), C.c_int64(stride), C.c_int32(out_rows),
        _p(feat_out, C.c_uint16), _p(tok_out, C.c_int32))
    if rc:
        raise ValueError("oracle_feature_gather failed: %d" % rc)
    return feat_out, tok_out

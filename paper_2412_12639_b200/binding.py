"""ctypes binding of libfalcon.so: same names as include/falcon.h, argument
marshalling only.  Every step of the verification path runs in the library's
CUDA kernels; there is no Python or CPU fallback, and loading fails loudly when
the shared library has not been built.

Tensors are passed as raw device addresses (``tensor.data_ptr()``); PyTorch is
used by callers only to own device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

T_MAX = 128
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_BAD_TREE, ERR_CAPACITY, ERR_TIMEOUT = range(7)
DEV_BAD_TREE, DEV_CAPACITY, DEV_BAD_PATH, DEV_TIMEOUT = 1, 2, 4, 8
ATTN_AUTO, ATTN_SIMT, ATTN_TC, ATTN_TCK, ATTN_WARP = 0, 1, 2, 3, 4
ATTN_PREFIX_STABLE = 1
ATTN_TEST_STALL = 1 << 30

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libfalcon.so")


class FalconError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = "%s failed: %s (%d)" % (where, status_string(code), code)
        super().__init__(msg + (": " + detail if detail else ""))


class TreeDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("total_nodes", C.c_int32), ("max_tree", C.c_int32),
                ("max_prefix_len", C.c_int32), ("node_off", C.c_void_p), ("parent", C.c_void_p),
                ("token", C.c_void_p), ("prefix_len", C.c_void_p), ("prefix_len_host", C.c_void_p),
                ("node_off_host", C.c_void_p), ("status", C.c_void_p)]


class AttnArgs(C.Structure):
    _fields_ = [("tree", TreeDesc), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("sm_scale", C.c_float), ("q", C.c_void_p), ("out", C.c_void_p), ("k_cache", C.c_void_p),
                ("v_cache", C.c_void_p), ("kv_stride_b", C.c_int64), ("kv_stride_h", C.c_int64),
                ("kv_stride_s", C.c_int64), ("s_cap", C.c_int32), ("k_tree", C.c_void_p), ("v_tree", C.c_void_p),
                ("tree_mask", C.c_void_p), ("kernel", C.c_int32), ("n_splits", C.c_int32), ("flags", C.c_int32),
                ("next_k_cache", C.c_void_p), ("next_v_cache", C.c_void_p)]


class AcceptArgs(C.Structure):
    _fields_ = [("tree", TreeDesc), ("vocab", C.c_int32), ("logits_stride", C.c_int64), ("logits", C.c_void_p),
                ("argmax_out", C.c_void_p), ("path", C.c_void_p), ("path_stride", C.c_int32),
                ("n_path", C.c_void_p), ("next_token", C.c_void_p), ("temperature", C.c_float),
                ("uniforms", C.c_void_p)]


class TopmArgs(C.Structure):
    _fields_ = [("n_rows", C.c_int32), ("vocab", C.c_int32), ("logits_stride", C.c_int64), ("logits", C.c_void_p),
                ("m", C.c_int32), ("top_val", C.c_void_p), ("top_idx", C.c_void_p)]


class LmArgmaxArgs(C.Structure):
    _fields_ = [("n_rows", C.c_int32), ("hidden", C.c_int32), ("vocab", C.c_int32), ("features", C.c_void_p),
                ("feat_stride", C.c_int64), ("lm_head", C.c_void_p), ("head_stride", C.c_int64),
                ("argmax_out", C.c_void_p), ("max_out", C.c_void_p), ("status", C.c_void_p), ("flags", C.c_int32)]


class GatherArgs(C.Structure):
    _fields_ = [("tree", TreeDesc), ("hidden", C.c_int32), ("feat_stride", C.c_int64), ("features", C.c_void_p),
                ("path", C.c_void_p), ("path_stride", C.c_int32), ("n_path", C.c_void_p), ("out_rows", C.c_int32),
                ("features_out", C.c_void_p), ("tokens_out", C.c_void_p)]


class CompactArgs(C.Structure):
    _fields_ = [("tree", TreeDesc), ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("k_cache_layers", C.c_void_p), ("v_cache_layers", C.c_void_p), ("kv_stride_b", C.c_int64),
                ("kv_stride_h", C.c_int64), ("kv_stride_s", C.c_int64), ("s_cap", C.c_int32),
                ("k_tree_layers", C.c_void_p), ("v_tree_layers", C.c_void_p), ("path", C.c_void_p),
                ("path_stride", C.c_int32), ("n_path", C.c_void_p), ("new_len", C.c_void_p),
                ("gather", C.POINTER(GatherArgs))]


_lib = None


def load_library():
    """Loads libfalcon.so; raises if it is missing (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            "%s not found: build it with `python -m paper_2412_12639_b200.build` (nvcc, sm_100a)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    lib.falcon_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    lib.falcon_create.restype = C.c_int
    lib.falcon_destroy.argtypes = [C.c_void_p]
    lib.falcon_destroy.restype = C.c_int
    lib.falcon_status_string.argtypes = [C.c_int]
    lib.falcon_status_string.restype = C.c_char_p
    lib.falcon_last_error.argtypes = [C.c_void_p]
    lib.falcon_last_error.restype = C.c_char_p
    lib.falcon_tree_validate_host.argtypes = [C.c_void_p, C.c_int32]
    lib.falcon_tree_validate_host.restype = C.c_int
    for name, argt in (("falcon_tree_attn", AttnArgs), ("falcon_tree_accept", AcceptArgs),
                       ("falcon_kv_compact", CompactArgs), ("falcon_topm", TopmArgs),
                       ("falcon_feature_gather", GatherArgs), ("falcon_lm_head_argmax", LmArgmaxArgs)):
        fn = getattr(lib, name)
        fn.argtypes = [C.c_void_p, C.POINTER(argt), C.c_void_p]
        fn.restype = C.c_int
    lib.falcon_test_poison.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
    lib.falcon_test_poison.restype = C.c_int
    lib.falcon_tree_attn_kernel.argtypes = [C.c_void_p, C.POINTER(AttnArgs)]
    lib.falcon_tree_attn_kernel.restype = C.c_int
    lib.falcon_tree_accept_static.argtypes = [C.POINTER(AcceptArgs), C.c_void_p]
    lib.falcon_tree_accept_static.restype = C.c_int
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().falcon_status_string(code).decode()


def falcon_tree_validate_host(parent) -> int:
    """parent: host int32 array of one tree.  Returns the status code."""
    import numpy as np
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    return int(load_library().falcon_tree_validate_host(parent.ctypes.data, len(parent)))


STATIC_MAX_NODES, STATIC_MAX_BATCH = 1024, 256
TOPM_MAX = 32
LM_TEST_STALL = 1 << 30


def falcon_tree_accept_static(args: "AcceptArgs", stream=None, check: bool = True) -> int:
    """Greedy acceptance without any device allocation: no context, scratch in a fixed array
    inside the library (limits STATIC_MAX_NODES / STATIC_MAX_BATCH).  For hosts that may not
    call cudaMalloc; calls that overlap on the GPU must be serialised by the caller."""
    rc = load_library().falcon_tree_accept_static(C.byref(args), _stream(stream))
    if check and rc:
        raise FalconError(rc, "falcon_tree_accept_static")
    return rc


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def tree_desc(batch, total_nodes, max_tree, max_prefix_len, node_off, parent, prefix_len, token=None,
              prefix_len_host=None, node_off_host=None, status=None) -> TreeDesc:
    """prefix_len_host / node_off_host: optional host int32 numpy arrays (kept alive by the caller)."""
    def host(a):
        return None if a is None else a.ctypes.data
    return TreeDesc(batch, total_nodes, max_tree, max_prefix_len, _ptr(node_off), _ptr(parent), _ptr(token),
                    _ptr(prefix_len), host(prefix_len_host), host(node_off_host), _ptr(status))


class Context:
    """Owns a falcon_ctx on one device."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        h = C.c_void_p()
        rc = self._lib.falcon_create(C.byref(h), device)
        if rc:
            raise FalconError(rc, "falcon_create")
        self._h = h
        self.device = device

    def close(self):
        if getattr(self, "_h", None):
            self._lib.falcon_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc:
            raise FalconError(rc, where, self._lib.falcon_last_error(self._h).decode())

    def falcon_tree_attn(self, args: AttnArgs, stream=None, check: bool = True) -> int:
        rc = self._lib.falcon_tree_attn(self._h, C.byref(args), _stream(stream))
        if check:
            self._check(rc, "falcon_tree_attn")
        return rc

    def falcon_tree_attn_kernel(self, args: AttnArgs) -> int:
        """The kernel (ATTN_SIMT / ATTN_TC / ATTN_TCK) falcon_tree_attn would run for `args`, -1 if it would refuse."""
        return int(self._lib.falcon_tree_attn_kernel(self._h, C.byref(args)))

    def falcon_tree_accept(self, args: AcceptArgs, stream=None, check: bool = True) -> int:
        rc = self._lib.falcon_tree_accept(self._h, C.byref(args), _stream(stream))
        if check:
            self._check(rc, "falcon_tree_accept")
        return rc

    def falcon_topm(self, args: TopmArgs, stream=None, check: bool = True) -> int:
        rc = self._lib.falcon_topm(self._h, C.byref(args), _stream(stream))
        if check:
            self._check(rc, "falcon_topm")
        return rc

    def falcon_lm_head_argmax(self, args: LmArgmaxArgs, stream=None, check: bool = True) -> int:
        rc = self._lib.falcon_lm_head_argmax(self._h, C.byref(args), _stream(stream))
        if check:
            self._check(rc, "falcon_lm_head_argmax")
        return rc

    def falcon_test_poison(self, pattern: int = 0xFFFFFFFF, stream=None) -> int:
        """Test hook: every SM's shared and tensor memory filled with `pattern`."""
        rc = self._lib.falcon_test_poison(self._h, pattern, _stream(stream))
        self._check(rc, "falcon_test_poison")
        return rc

    def falcon_feature_gather(self, args: GatherArgs, stream=None, check: bool = True) -> int:
        rc = self._lib.falcon_feature_gather(self._h, C.byref(args), _stream(stream))
        if check:
            self._check(rc, "falcon_feature_gather")
        return rc

    def falcon_kv_compact(self, args: CompactArgs, stream=None, check: bool = True) -> int:
        rc = self._lib.falcon_kv_compact(self._h, C.byref(args), _stream(stream))
        if check:
            self._check(rc, "falcon_kv_compact")
        return rc


def attn_args(tree: TreeDesc, n_q_heads, n_kv_heads, head_dim, sm_scale, q, out, k_cache, v_cache, strides, s_cap,
              k_tree=None, v_tree=None, tree_mask=None, kernel=ATTN_AUTO, n_splits=0, flags=0,
              next_k_cache=None, next_v_cache=None) -> AttnArgs:
    """flags: ATTN_PREFIX_STABLE when the prefix rows were written before the preceding kernel started.
    next_k_cache / next_v_cache: the caches the next call on the stream will read (an L2 prefetch hint)."""
    return AttnArgs(tree, n_q_heads, n_kv_heads, head_dim, sm_scale, _ptr(q), _ptr(out), _ptr(k_cache),
                    _ptr(v_cache), strides[0], strides[1], strides[2], s_cap, _ptr(k_tree), _ptr(v_tree),
                    _ptr(tree_mask), kernel, n_splits, flags, _ptr(next_k_cache), _ptr(next_v_cache))


def accept_args(tree: TreeDesc, vocab, logits, logits_stride, argmax_out, path, path_stride, n_path,
                next_token, temperature: float = 0.0, uniforms=None) -> AcceptArgs:
    """temperature > 0: the nodes' tokens are drawn from softmax(logits / temperature) with `uniforms` [N]."""
    return AcceptArgs(tree, vocab, logits_stride, _ptr(logits), _ptr(argmax_out), _ptr(path), path_stride,
                      _ptr(n_path), _ptr(next_token), temperature, _ptr(uniforms))


def topm_args(n_rows, vocab, logits, logits_stride, m, top_val, top_idx) -> TopmArgs:
    return TopmArgs(n_rows, vocab, logits_stride, _ptr(logits), m, _ptr(top_val), _ptr(top_idx))


def lm_argmax_args(n_rows, hidden, vocab, features, feat_stride, lm_head, head_stride, argmax_out, max_out=None,
                   status=None, flags=0) -> LmArgmaxArgs:
    return LmArgmaxArgs(n_rows, hidden, vocab, _ptr(features), feat_stride, _ptr(lm_head), head_stride,
                        _ptr(argmax_out), _ptr(max_out), _ptr(status), flags)


def gather_args(tree: TreeDesc, hidden, features, feat_stride, path, path_stride, n_path, out_rows, features_out,
                tokens_out) -> GatherArgs:
    return GatherArgs(tree, hidden, feat_stride, _ptr(features), _ptr(path), path_stride, _ptr(n_path), out_rows,
                      _ptr(features_out), _ptr(tokens_out))


def compact_args(tree: TreeDesc, n_layers, n_kv_heads, head_dim, k_cache_layers, v_cache_layers, strides, s_cap,
                 path, path_stride, n_path, new_len, k_tree_layers=None, v_tree_layers=None,
                 gather: Optional[GatherArgs] = None) -> CompactArgs:
    """gather: record the accepted tokens and features in the same launch (the caller keeps `gather` alive
    until the call has returned)."""
    return CompactArgs(tree, n_layers, n_kv_heads, head_dim, _ptr(k_cache_layers), _ptr(v_cache_layers),
                       strides[0], strides[1], strides[2], s_cap, _ptr(k_tree_layers), _ptr(v_tree_layers),
                       _ptr(path), path_stride, _ptr(n_path), _ptr(new_len),
                       C.pointer(gather) if gather is not None else None)
